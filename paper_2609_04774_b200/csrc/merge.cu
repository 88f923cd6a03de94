// cp_merge: N-way log-sum-exp combination of partial attention results.  HBM-bound streaming
// kernel: one warp per (token, head) row of 128 floats, each lane owning one float4 of the row.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"

using namespace cpattn;

namespace {

constexpr int kMergeD = 128;
constexpr int kTokPerCta = 8;    // tokens per CTA: 8 consecutive lse floats = one 32-byte sector
constexpr int kMergeThreads = 32 * kTokPerCta;

__device__ __forceinline__ float4 ld_stream(const float4* p) {
    float4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
    return v;
}

// Grid: one-dimensional, block b = y * gx + x with gx = ceil(H / HPW), y < ceil(T / kTokPerCta) (consecutive
// blocks read consecutive memory).  Warp w of the CTA handles token y*8 + w and heads
// x*HPW .. x*HPW+HPW-1 (HPW consecutive rows of every partial, 512 B each).  N <= NMAX; all HPW*NMAX
// row loads of a warp are issued before the first use so that enough bytes are in flight per SM.
template <int NMAX, int HPW, bool kOutBf16>
__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const float* __restrict__ partials, const float* __restrict__ lses, int N, int64_t T, int H, int gx,
             void* __restrict__ out, float* __restrict__ lse_out) {
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int64_t t = (int64_t)(blockIdx.x / gx) * kTokPerCta + warp;
    const int h0 = (blockIdx.x % gx) * HPW;
    if (t >= T) return;
    const int64_t row_stride4 = kMergeD / 4;                          // float4 per row
    const int64_t part_stride4 = T * (int64_t)H * row_stride4;        // float4 per partial
    const float4* src = reinterpret_cast<const float4*>(partials) + (t * H + h0) * row_stride4 + lane;

    float4 x[HPW][NMAX];
    float my[HPW];
#pragma unroll
    for (int hh = 0; hh < HPW; ++hh) {
        const bool hv = h0 + hh < H;
        // lane n < N holds lse of partial n
        my[hh] = (hv && lane < N) ? lses[((int64_t)lane * H + h0 + hh) * T + t] : -INFINITY;
#pragma unroll
        for (int n = 0; n < NMAX; ++n)
            if (hv && n < N) x[hh][n] = ld_stream(src + n * part_stride4 + hh * row_stride4);
    }
#pragma unroll
    for (int hh = 0; hh < HPW; ++hh) {
        const int h = h0 + hh;
        if (h >= H) break;
        // max / sum of the partial LSEs by warp shuffles
        float m = my[hh];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
        const bool dead = (m == -INFINITY);
        const float w = (dead || my[hh] == -INFINITY) ? 0.f : __expf(my[hh] - m);
        float ws = w;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ws += __shfl_xor_sync(0xffffffffu, ws, o);
        const float inv = dead ? 0.f : 1.f / ws;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int n = 0; n < NMAX; ++n) {
            if (n < N) {
                const float wn = __shfl_sync(0xffffffffu, w, n) * inv;
                if (wn > 0.f) {   // a zero weight hides whatever the partial holds
                    acc.x = fmaf(wn, x[hh][n].x, acc.x);
                    acc.y = fmaf(wn, x[hh][n].y, acc.y);
                    acc.z = fmaf(wn, x[hh][n].z, acc.z);
                    acc.w = fmaf(wn, x[hh][n].w, acc.w);
                }
            }
        }
        const int64_t orow = (t * H + h) * kMergeD + lane * 4;
        if (kOutBf16) {
            __nv_bfloat162 a = __floats2bfloat162_rn(acc.x, acc.y);
            __nv_bfloat162 b = __floats2bfloat162_rn(acc.z, acc.w);
            uint2 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&a);
            pk.y = *reinterpret_cast<uint32_t*>(&b);
            __stcs(reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(out) + orow), pk);
        } else {
            __stcs(reinterpret_cast<float4*>(reinterpret_cast<float*>(out) + orow), acc);
        }
        if (lse_out != nullptr && lane == 0) lse_out[(int64_t)h * T + t] = dead ? -INFINITY : m + __logf(ws);
    }
}

template <int NMAX, int HPW>
void launch_merge(const float* partials, const float* lses, int N, int64_t T, int H, void* out, int out_dtype,
                  float* lse_out, cudaStream_t s) {
    const int gx = (H + HPW - 1) / HPW;
    const unsigned grid = (unsigned)(gx * ((T + kTokPerCta - 1) / kTokPerCta));
    if (out_dtype == CP_DTYPE_BF16)
        merge_kernel<NMAX, HPW, true><<<grid, kMergeThreads, 0, s>>>(partials, lses, N, T, H, gx, out, lse_out);
    else
        merge_kernel<NMAX, HPW, false><<<grid, kMergeThreads, 0, s>>>(partials, lses, N, T, H, gx, out, lse_out);
}

}  // namespace

extern "C" int cp_merge(cp_ctx* ctx, const float* partials, const float* lses, int32_t N, int64_t T, int32_t H,
                        int32_t D, void* out, int32_t out_dtype, float* lse_out, void* stream) {
    if (!ctx || !partials || !lses || !out || N < 1 || T < 1 || H < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_merge: null pointer or non-positive size (N=%d T=%lld H=%d)", N,
                         (long long)T, H);
    if (D != kMergeD) return set_error(CP_ERR_UNSUPPORTED, "cp_merge: D=%d, only 128 is supported", D);
    if (N > 32) return set_error(CP_ERR_UNSUPPORTED, "cp_merge: N=%d, at most 32 partials", N);
    if (out_dtype != CP_DTYPE_BF16 && out_dtype != CP_DTYPE_F32)
        return set_error(CP_ERR_INVALID_ARG, "cp_merge: out_dtype=%d", out_dtype);
    if ((T + kTokPerCta - 1) / kTokPerCta * (int64_t)H > 0x7fffffffll)
        return set_error(CP_ERR_UNSUPPORTED, "cp_merge: T=%lld x H=%d needs more than 2^31 blocks", (long long)T, H);
    if (((uintptr_t)partials | (uintptr_t)out) & 15)
        return set_error(CP_ERR_INVALID_ARG, "cp_merge: partials and out must be 16-byte aligned");
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // heads per warp: measured.  Two partials: 2 heads per warp (4 row loads in flight per warp, many warps)
    // reach 6.2-6.6 TB/s where 4 heads gave 5.9-6.1 and 8 heads 4.4; one head per warp loses 10 %.  The output
    // rows are written once and never re-read: streaming stores keep them from displacing input lines in L2.
    if (N <= 2) launch_merge<2, 2>(partials, lses, N, T, H, out, out_dtype, lse_out, s);
    else if (N <= 4) launch_merge<4, 2>(partials, lses, N, T, H, out, out_dtype, lse_out, s);
    else if (N <= 8) launch_merge<8, 1>(partials, lses, N, T, H, out, out_dtype, lse_out, s);
    else if (N <= 16) launch_merge<16, 1>(partials, lses, N, T, H, out, out_dtype, lse_out, s);
    else launch_merge<32, 1>(partials, lses, N, T, H, out, out_dtype, lse_out, s);
    return check_cuda(cudaGetLastError(), "cp_merge launch");
}

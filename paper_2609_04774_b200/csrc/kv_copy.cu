// cp_kv_gather / cp_kv_append: bit-exact copies between a paged KV cache and contiguous rows,
// addressed through the page table.  One 16-byte vector per thread; HBM-bound.
#include <cuda_bf16.h>

#include <algorithm>

#include "internal.h"

using namespace cpattn;

namespace {

// One token's row of vec_per_tok 16-byte vectors, copied by one warp: four vectors per lane and tensor are in flight
// before the first store.  `paged` is the address of the token's slot (head 0, vector 0); head g starts
// stride_head8 vectors further.  vph_shift = log2(vectors per head row): 4 (bf16) or 3 (one-byte elements).
template <bool kToPaged>
__device__ __forceinline__ void copy_token(uint4* __restrict__ paged_k, uint4* __restrict__ paged_v, uint4* __restrict__ rows_k,
                                           uint4* __restrict__ rows_v, int64_t paged_off, int64_t rows_off, int vec_per_tok,
                                           int vph_shift, int64_t stride_head8, int lane) {
    for (int v0 = 0; v0 < vec_per_tok; v0 += 128) {
        int64_t po[4];
        uint4 a[4], b[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int v = v0 + u * 32 + lane;
            const int g = v >> vph_shift;
            po[u] = paged_off + (int64_t)g * stride_head8 + (v - (g << vph_shift));
            if (v < vec_per_tok) {
                if (rows_k) a[u] = kToPaged ? rows_k[rows_off + v] : paged_k[po[u]];
                if (rows_v) b[u] = kToPaged ? rows_v[rows_off + v] : paged_v[po[u]];
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int v = v0 + u * 32 + lane;
            if (v < vec_per_tok) {
                if (kToPaged) {
                    if (rows_k) paged_k[po[u]] = a[u];
                    if (rows_v) paged_v[po[u]] = b[u];
                } else {
                    if (rows_k) rows_k[rows_off + v] = a[u];
                    if (rows_v) rows_v[rows_off + v] = b[u];
                }
            }
        }
    }
}

// Records the first page id outside the pool in the status words {code, table index, block, page id}.
__device__ __forceinline__ void report_bad_page(int32_t* status, int64_t table_index, int64_t page) {
    if (atomicCAS(status, 0, CP_ERR_BOUNDS) == 0) {
        status[1] = (int32_t)table_index;
        status[2] = (int32_t)blockIdx.x;
        status[3] = (int32_t)page;
    }
}

// kToPaged = false: paged -> rows (gather); true: rows -> paged (append).  One warp per token (the page id is looked up
// once per token); page_shift = log2(page_size).
template <bool kToPaged>
__global__ void __launch_bounds__(256)
kv_copy_kernel(uint4* __restrict__ paged_k, uint4* __restrict__ paged_v, uint4* __restrict__ rows_k,
               uint4* __restrict__ rows_v, const int32_t* __restrict__ page_table, int64_t t_begin, int64_t n,
               int page_shift, int Hkv, int vph_shift, int64_t stride_page8, int64_t stride_tok8,
               int64_t stride_head8, int64_t num_pages, int32_t* status) {
    const int vec_per_tok = Hkv << vph_shift;
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t tok = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; tok < n; tok += n_warps) {
        const int64_t t = t_begin + tok;
        const int64_t page = page_table[t >> page_shift];
        if (page < 0 || page >= num_pages) {
            // a page id outside the pool: the token is skipped (nothing is read or written through it)
            if (lane == 0) report_bad_page(status, t >> page_shift, page);
            continue;
        }
        copy_token<kToPaged>(paged_k, paged_v, rows_k, rows_v,
                             page * stride_page8 + (t & ((1ll << page_shift) - 1)) * stride_tok8, tok * vec_per_tok, vec_per_tok,
                             vph_shift, stride_head8, lane);
    }
}

// page sizes are powers of two (validate_cache): log2
inline int log2_of(int v) {
    int s = 0;
    while ((1 << s) < v) ++s;
    return s;
}

int validate_cache(const cp_kv_cache* c, const char* who) {
    if (!c || !c->k || !c->v || c->num_pages < 1 || c->Hkv < 1)
        return set_error(CP_ERR_INVALID_ARG, "%s: cache is NULL or has null / non-positive fields", who);
    if ((c->page_size != 16 && c->page_size != 32 && c->page_size != 64 && c->page_size != 128) || c->D != 128)
        return set_error(CP_ERR_UNSUPPORTED, "%s: page_size=%d D=%d; supported: pages of 16, 32, 64 or 128 tokens, D = 128", who,
                         c->page_size, c->D);
    if ((c->stride_page | c->stride_tok | c->stride_head) & 7 || c->stride_page < 1 || c->stride_tok < 1 ||
        c->stride_head < 1)
        return set_error(CP_ERR_UNSUPPORTED, "%s: strides must be positive multiples of 8 elements", who);
    if (((uintptr_t)c->k | (uintptr_t)c->v) & 15)
        return set_error(CP_ERR_UNSUPPORTED, "%s: k and v must be 16-byte aligned", who);
    return CP_OK;
}

// Several runs of rows in one launch: segment i writes rows [row0, row0 + n) of the row buffers to logical tokens
// [t_begin, t_begin + n).  The segment table travels in the launch parameters.
constexpr int kMaxSegments = 64;
struct SegmentTable {
    int32_t n_segments;
    int64_t t_begin[kMaxSegments];
    int64_t row0[kMaxSegments];
    int64_t cum[kMaxSegments + 1];     // prefix sums of the segment lengths
};

__global__ void __launch_bounds__(256)
kv_append_segments_kernel(uint4* __restrict__ paged_k, uint4* __restrict__ paged_v, const uint4* __restrict__ rows_k,
                          const uint4* __restrict__ rows_v, const int32_t* __restrict__ page_table,
                          const __grid_constant__ SegmentTable seg, int page_shift, int Hkv, int vph_shift,
                          int64_t stride_page8, int64_t stride_tok8, int64_t stride_head8, int64_t num_pages,
                          int32_t* status) {
    const int vec_per_tok = Hkv << vph_shift;
    const int lane = threadIdx.x & 31;
    const int64_t n = seg.cum[seg.n_segments];
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    int sg = 0;
    for (int64_t tok = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; tok < n; tok += n_warps) {
        while (tok >= seg.cum[sg + 1]) ++sg;                       // tokens ascend: the walk never goes back
        const int64_t k = tok - seg.cum[sg];
        const int64_t t = seg.t_begin[sg] + k;
        const int64_t page = page_table[t >> page_shift];
        if (page < 0 || page >= num_pages) {
            if (lane == 0) report_bad_page(status, t >> page_shift, page);
            continue;
        }
        copy_token<true>(paged_k, paged_v, const_cast<uint4*>(rows_k), const_cast<uint4*>(rows_v),
                         page * stride_page8 + (t & ((1ll << page_shift) - 1)) * stride_tok8, (seg.row0[sg] + k) * vec_per_tok,
                         vec_per_tok, vph_shift, stride_head8, lane);
    }
}

// Debug aid: every entry of a device page table against the pool size.  The table is only read, never used as an
// address; the first entry outside [0, num_pages) lands in the status words {code, index, block, page id}.
__global__ void __launch_bounds__(256)
check_page_table_kernel(const int32_t* __restrict__ page_table, int64_t n, int64_t num_pages, int32_t* status) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        const int64_t page = page_table[i];
        if ((page < 0 || page >= num_pages) && atomicCAS(status, 0, CP_ERR_BOUNDS) == 0) {
            status[1] = (int32_t)i;
            status[2] = (int32_t)blockIdx.x;
            status[3] = (int32_t)page;
        }
    }
}

// FP8 cache writer: eight bf16 values of a row -> eight E4M3 bytes, each e4m3_rne_satfinite(x / scale[g]) with
// the quotient rounded to fp32 first.  Page ids outside the pool are skipped and reported like in the copies.
__device__ __forceinline__ uint32_t quant4(float a, float b, float c, float d, float sc) {
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(__fdiv_rn(b, sc)), "f"(__fdiv_rn(a, sc)));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(__fdiv_rn(d, sc)), "f"(__fdiv_rn(c, sc)));
    return (uint32_t)lo | ((uint32_t)hi << 16);
}

__global__ void __launch_bounds__(256)
kv_append_fp8_kernel(uint8_t* __restrict__ paged_k, uint8_t* __restrict__ paged_v, const uint4* __restrict__ rows_k,
                     const uint4* __restrict__ rows_v, const float* __restrict__ k_scale, const float* __restrict__ v_scale,
                     const int32_t* __restrict__ page_table, int64_t t_begin, int64_t n, int page_shift, int Hkv,
                     int64_t stride_page, int64_t stride_tok, int64_t stride_head, int64_t num_pages, int32_t* status) {
    const int vec_per_tok = Hkv * 16;                 // one warp per token, 8 elements (16 bytes in, 8 bytes out) per lane and step
    const int lane = threadIdx.x & 31;
    const int64_t n_warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t tok = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; tok < n; tok += n_warps) {
        const int64_t t = t_begin + tok;
        const int64_t page = page_table[t >> page_shift];
        if (page < 0 || page >= num_pages) {
            if (lane == 0) report_bad_page(status, t >> page_shift, page);
            continue;
        }
        const int64_t tok_off = page * stride_page + (t & ((1ll << page_shift) - 1)) * stride_tok;
        for (int v = lane; v < vec_per_tok; v += 32) {
            const int g = v >> 4, c = v & 15;
            const int64_t off = tok_off + (int64_t)g * stride_head + c * 8;
#pragma unroll
            for (int kv = 0; kv < 2; ++kv) {
                const uint4* rows = kv ? rows_v : rows_k;
                if (!rows) continue;
                const uint4 raw = rows[tok * vec_per_tok + v];
                const float sc = kv ? v_scale[g] : k_scale[g];
                const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&raw);
                uint2 o;
                o.x = quant4(__low2float(h[0]), __high2float(h[0]), __low2float(h[1]), __high2float(h[1]), sc);
                o.y = quant4(__low2float(h[2]), __high2float(h[2]), __low2float(h[3]), __high2float(h[3]), sc);
                *reinterpret_cast<uint2*>((kv ? paged_v : paged_k) + off) = o;
            }
        }
    }
}

int validate_cache_fp8(const cp_kv_cache_fp8* c, const char* who) {
    if (!c || !c->k || !c->v || !c->k_scale || !c->v_scale || c->num_pages < 1 || c->Hkv < 1)
        return set_error(CP_ERR_INVALID_ARG, "%s: FP8 cache is NULL or has null / non-positive fields", who);
    if ((c->page_size != 16 && c->page_size != 32 && c->page_size != 64 && c->page_size != 128) || c->D != 128)
        return set_error(CP_ERR_UNSUPPORTED, "%s: page_size=%d D=%d; supported: pages of 16, 32, 64 or 128 tokens, D = 128", who,
                         c->page_size, c->D);
    if ((c->stride_page | c->stride_tok | c->stride_head) & 15 || c->stride_page < 1 || c->stride_tok < 1 ||
        c->stride_head < 1)
        return set_error(CP_ERR_UNSUPPORTED, "%s: FP8 cache strides must be positive multiples of 16 bytes", who);
    if (((uintptr_t)c->k | (uintptr_t)c->v) & 15)
        return set_error(CP_ERR_UNSUPPORTED, "%s: k and v must be 16-byte aligned", who);
    return CP_OK;
}

template <bool kToPaged>
int kv_copy(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int64_t t_begin, int64_t n,
            const void* k_rows, const void* v_rows, void* stream, const char* who) {
    if (!ctx || !page_table || t_begin < 0 || n < 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer or negative range", who);
    if (int rc = validate_cache(cache, who)) return rc;
    if (!k_rows && !v_rows) return set_error(CP_ERR_INVALID_ARG, "%s: both row pointers are NULL", who);
    if (((uintptr_t)k_rows | (uintptr_t)v_rows) & 15)
        return set_error(CP_ERR_INVALID_ARG, "%s: row buffers must be 16-byte aligned", who);
    if (n == 0) return CP_OK;
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    const int blocks = (int)std::min<int64_t>((n + 7) / 8, (int64_t)ctx->num_sms * 16);      // one warp per token
    kv_copy_kernel<kToPaged><<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        (uint4*)cache->k, (uint4*)cache->v, (uint4*)k_rows, (uint4*)v_rows, page_table, t_begin, n, log2_of(cache->page_size),
        cache->Hkv, 4, cache->stride_page / 8, cache->stride_tok / 8, cache->stride_head / 8, cache->num_pages,
        ctx->d_status);
    return check_cuda(cudaGetLastError(), who);
}

// The segment form for both cache kinds: `elem_shift` = log2(bytes per element) turns the caller's strides into
// 16-byte vectors (bf16: strides in elements, 8 per vector; one-byte elements: strides in bytes, 16 per vector).
int append_segments(cp_ctx* ctx, void* cache_k, void* cache_v, int32_t page_size, int32_t Hkv, int64_t stride_page,
                    int64_t stride_tok, int64_t stride_head, int64_t num_pages, bool one_byte, const int32_t* page_table,
                    int32_t n_segments, const cp_kv_segment* segments, const void* k_rows, const void* v_rows, void* stream,
                    const char* who) {
    if (!k_rows && !v_rows) return set_error(CP_ERR_INVALID_ARG, "%s: both row pointers are NULL", who);
    if (((uintptr_t)k_rows | (uintptr_t)v_rows) & 15)
        return set_error(CP_ERR_INVALID_ARG, "%s: row buffers must be 16-byte aligned", who);
    SegmentTable tab;
    tab.n_segments = 0;
    tab.cum[0] = 0;
    for (int32_t i = 0; i < n_segments; ++i) {
        const cp_kv_segment& sg = segments[i];
        if (sg.t_begin < 0 || sg.n < 0 || sg.row0 < 0)
            return set_error(CP_ERR_INVALID_ARG, "%s: segment %d has a negative field", who, i);
        if (sg.n == 0) continue;
        const int k = tab.n_segments++;
        tab.t_begin[k] = sg.t_begin;
        tab.row0[k] = sg.row0;
        tab.cum[k + 1] = tab.cum[k] + sg.n;
    }
    if (tab.n_segments == 0) return CP_OK;
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    const int per_vec = one_byte ? 16 : 8;          // stride units per 16-byte vector
    const int blocks = (int)std::min<int64_t>((tab.cum[tab.n_segments] + 7) / 8, (int64_t)ctx->num_sms * 16);   // one warp per token
    kv_append_segments_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        (uint4*)cache_k, (uint4*)cache_v, (const uint4*)k_rows, (const uint4*)v_rows, page_table, tab, log2_of(page_size), Hkv,
        one_byte ? 3 : 4, stride_page / per_vec, stride_tok / per_vec, stride_head / per_vec, num_pages, ctx->d_status);
    return check_cuda(cudaGetLastError(), who);
}

}  // namespace

namespace cpattn {
int validate_kv_cache(const cp_kv_cache* c, const char* who) { return validate_cache(c, who); }
int validate_kv_cache_fp8(const cp_kv_cache_fp8* c, const char* who) { return validate_cache_fp8(c, who); }
}

extern "C" int cp_kv_append_segments(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int32_t n_segments,
                                     const cp_kv_segment* segments, const void* k_rows, const void* v_rows, void* stream) {
    const char* who = "cp_kv_append_segments";
    if (!ctx || !page_table || !segments || n_segments < 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer or negative segment count", who);
    if (n_segments > kMaxSegments)
        return set_error(CP_ERR_UNSUPPORTED, "%s: %d segments, at most %d per call", who, n_segments, kMaxSegments);
    if (int rc = validate_cache(cache, who)) return rc;
    return append_segments(ctx, const_cast<void*>(cache->k), const_cast<void*>(cache->v), cache->page_size, cache->Hkv, cache->stride_page, cache->stride_tok,
                           cache->stride_head, cache->num_pages, false, page_table, n_segments, segments, k_rows, v_rows, stream, who);
}

extern "C" int cp_check_page_table(cp_ctx* ctx, const int32_t* page_table, int64_t n_entries, int64_t num_pages, void* stream) {
    if (!ctx || !page_table || n_entries < 0 || num_pages < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_check_page_table: null pointer, negative count or empty pool");
    if (n_entries == 0) return CP_OK;
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    const int blocks = (int)std::min<int64_t>((n_entries + 255) / 256, (int64_t)ctx->num_sms * 8);
    check_page_table_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(page_table, n_entries, num_pages, ctx->d_status);
    return check_cuda(cudaGetLastError(), "cp_check_page_table");
}

// Raw byte copies of an FP8 cache (no conversion): the same kernels with one-byte elements, i.e. 8 vectors of 16
// bytes per head row.  What a CP rank exchanges when the cache is FP8: stored bytes travel, and because all ranks
// share the per-head scales they can be appended as they are.
extern "C" int cp_kv_gather_fp8(cp_ctx* ctx, const cp_kv_cache_fp8* cache, const int32_t* page_table, int64_t t_begin,
                                int64_t n, void* k_bytes, void* v_bytes, void* stream) {
    const char* who = "cp_kv_gather_fp8";
    if (!ctx || !page_table || t_begin < 0 || n < 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer or negative range", who);
    if (int rc = validate_cache_fp8(cache, who)) return rc;
    if (!k_bytes && !v_bytes) return set_error(CP_ERR_INVALID_ARG, "%s: both row pointers are NULL", who);
    if (((uintptr_t)k_bytes | (uintptr_t)v_bytes) & 15)
        return set_error(CP_ERR_INVALID_ARG, "%s: row buffers must be 16-byte aligned", who);
    if (n == 0) return CP_OK;
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    const int blocks = (int)std::min<int64_t>((n + 7) / 8, (int64_t)ctx->num_sms * 16);
    kv_copy_kernel<false><<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        (uint4*)cache->k, (uint4*)cache->v, (uint4*)k_bytes, (uint4*)v_bytes, page_table, t_begin, n, log2_of(cache->page_size),
        cache->Hkv, 3, cache->stride_page / 16, cache->stride_tok / 16, cache->stride_head / 16, cache->num_pages,
        ctx->d_status);
    return check_cuda(cudaGetLastError(), who);
}

extern "C" int cp_kv_append_segments_fp8(cp_ctx* ctx, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                                         int32_t n_segments, const cp_kv_segment* segments, const void* k_bytes,
                                         const void* v_bytes, void* stream) {
    const char* who = "cp_kv_append_segments_fp8";
    if (!ctx || !page_table || !segments || n_segments < 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer or negative segment count", who);
    if (n_segments > kMaxSegments)
        return set_error(CP_ERR_UNSUPPORTED, "%s: %d segments, at most %d per call", who, n_segments, kMaxSegments);
    if (int rc = validate_cache_fp8(cache, who)) return rc;
    return append_segments(ctx, const_cast<void*>(cache->k), const_cast<void*>(cache->v), cache->page_size, cache->Hkv,
                           cache->stride_page, cache->stride_tok, cache->stride_head, cache->num_pages, true, page_table,
                           n_segments, segments, k_bytes, v_bytes, stream, who);
}

extern "C" int cp_kv_append_fp8(cp_ctx* ctx, const cp_kv_cache_fp8* cache, const int32_t* page_table, int64_t t_begin,
                                int64_t n, const void* k_rows, const void* v_rows, void* stream) {
    const char* who = "cp_kv_append_fp8";
    if (!ctx || !page_table || t_begin < 0 || n < 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer or negative range", who);
    if (int rc = validate_cache_fp8(cache, who)) return rc;
    if (!k_rows && !v_rows) return set_error(CP_ERR_INVALID_ARG, "%s: both row pointers are NULL", who);
    if (((uintptr_t)k_rows | (uintptr_t)v_rows) & 15)
        return set_error(CP_ERR_INVALID_ARG, "%s: row buffers must be 16-byte aligned", who);
    if (n == 0) return CP_OK;
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    const int blocks = (int)std::min<int64_t>((n + 7) / 8, (int64_t)ctx->num_sms * 16);       // one warp per token
    kv_append_fp8_kernel<<<blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
        (uint8_t*)cache->k, (uint8_t*)cache->v, (const uint4*)k_rows, (const uint4*)v_rows, cache->k_scale, cache->v_scale,
        page_table, t_begin, n, log2_of(cache->page_size), cache->Hkv, cache->stride_page, cache->stride_tok, cache->stride_head,
        cache->num_pages, ctx->d_status);
    return check_cuda(cudaGetLastError(), who);
}

extern "C" int cp_kv_gather(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int64_t t_begin,
                            int64_t n, void* k_rows, void* v_rows, void* stream) {
    return kv_copy<false>(ctx, cache, page_table, t_begin, n, k_rows, v_rows, stream, "cp_kv_gather");
}

extern "C" int cp_kv_append(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int64_t t_begin,
                            int64_t n, const void* k_rows, const void* v_rows, void* stream) {
    return kv_copy<true>(ctx, cache, page_table, t_begin, n, k_rows, v_rows, stream, "cp_kv_append");
}

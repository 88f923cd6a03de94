// Host side of the attention calls of libcpattn: argument validation, the varlen tile schedule's upload (or its
// ride in the launch parameters), tensor maps, launches, and the C entry points.  The kernels themselves
// (cp_attn_kernel, the LSE fix-up of KV-split units, the fill of uncovered rows) are in attn_kernel.cuh.
#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "internal.h"
#include "attn_kernel.cuh"

using namespace cpattn;

namespace {

int encode_maps(cp_ctx* ctx, const void* q, int64_t total_rows, int32_t Hq, const cp_kv_cache* c, CUtensorMap* tmQ,
                CUtensorMap* tmK, CUtensorMap* tmV) {
    {
        cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)Hq, (cuuint64_t)total_rows};
        cuuint64_t strides[2] = {(cuuint64_t)kD * 2, (cuuint64_t)Hq * kD * 2};
        cuuint32_t box[3] = {64, 1, (cuuint32_t)kBlockM};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult r = ctx->encode_tiled(tmQ, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(q), dims, strides, box,
                                       es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return set_error(CP_ERR_CUDA, "cuTensorMapEncodeTiled(q) failed with %d", (int)r);
    }
    for (int kv = 0; kv < 2; ++kv) {
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)c->Hkv, (cuuint64_t)c->page_size, (cuuint64_t)c->num_pages};
        cuuint64_t strides[3] = {(cuuint64_t)c->stride_head * 2, (cuuint64_t)c->stride_tok * 2,
                                 (cuuint64_t)c->stride_page * 2};
        cuuint32_t box[4] = {64, 1, (cuuint32_t)c->page_size, 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        CUresult r = ctx->encode_tiled(kv ? tmV : tmK, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4,
                                       const_cast<void*>(kv ? c->v : c->k), dims, strides, box, es,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return set_error(CP_ERR_CUDA, "cuTensorMapEncodeTiled(%s) failed with %d", kv ? "v" : "k", (int)r);
    }
    return CP_OK;
}

// Tensor maps of the FP8 variant: one-byte elements, a 128-dim row is one 128-byte swizzle line.
int encode_maps_fp8(cp_ctx* ctx, const void* q8, int64_t total_rows, int32_t Hq, const cp_kv_cache_fp8* c, CUtensorMap* tmQ,
                    CUtensorMap* tmK, CUtensorMap* tmV) {
    {
        cuuint64_t dims[3] = {(cuuint64_t)kD, (cuuint64_t)Hq, (cuuint64_t)total_rows};
        cuuint64_t strides[2] = {(cuuint64_t)kD, (cuuint64_t)Hq * kD};
        cuuint32_t box[3] = {(cuuint32_t)kD, 1, (cuuint32_t)kBlockM};
        cuuint32_t es[3] = {1, 1, 1};
        CUresult r = ctx->encode_tiled(tmQ, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<void*>(q8), dims, strides, box,
                                       es, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return set_error(CP_ERR_CUDA, "cuTensorMapEncodeTiled(q8) failed with %d", (int)r);
    }
    for (int kv = 0; kv < 2; ++kv) {
        cuuint64_t dims[4] = {(cuuint64_t)kD, (cuuint64_t)c->Hkv, (cuuint64_t)c->page_size, (cuuint64_t)c->num_pages};
        cuuint64_t strides[3] = {(cuuint64_t)c->stride_head, (cuuint64_t)c->stride_tok, (cuuint64_t)c->stride_page};
        cuuint32_t box[4] = {(cuuint32_t)kD, 1, (cuuint32_t)c->page_size, 1};
        cuuint32_t es[4] = {1, 1, 1, 1};
        CUresult r = ctx->encode_tiled(kv ? tmV : tmK, CU_TENSOR_MAP_DATA_TYPE_UINT8, 4,
                                       const_cast<void*>(kv ? c->v : c->k), dims, strides, box, es,
                                       CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                                       CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return set_error(CP_ERR_CUDA, "cuTensorMapEncodeTiled(%s8) failed with %d", kv ? "v" : "k", (int)r);
    }
    return CP_OK;
}

// Query quantisation of the FP8 variant, one warp per (token, head) row of 128 bf16 values: amax by shuffles,
// q_scale = amax / 448 and inv = 448 / amax (IEEE divisions), code = e4m3(q * inv) with round to nearest even and
// saturation; a row of zeros gets scale 0 and codes 0.
__global__ void __launch_bounds__(256)
quantize_q_kernel(const __nv_bfloat16* __restrict__ q, uint8_t* __restrict__ q8, float* __restrict__ q_scale, int64_t n_rows) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    if (row >= n_rows) return;
    const uint2 raw = reinterpret_cast<const uint2*>(q + row * kD)[lane];
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    const float x0 = __low2float(a), x1 = __high2float(a), x2 = __low2float(b), x3 = __high2float(b);
    float amax = fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3)));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    const float inv = amax > 0.f ? __fdiv_rn(448.f, amax) : 0.f;
    reinterpret_cast<uint32_t*>(q8 + row * kD)[lane] =
        pack_e4m3x4(__fmul_rn(x0, inv), __fmul_rn(x1, inv), __fmul_rn(x2, inv), __fmul_rn(x3, inv));
    if (lane == 0) q_scale[row] = amax > 0.f ? __fdiv_rn(amax, 448.f) : 0.f;
}

// Moves 16-byte words from pinned host memory (read over PCIe) into device memory.  Used instead of a
// copy-engine transfer for the schedule: a kernel stays on the compute engine, so the attention launch
// behind it does not wait on a cross-engine hand-over.
__global__ void stage_copy_kernel(uint4* __restrict__ dst, const uint4* __restrict__ src, int64_t n16) {
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (int64_t)gridDim.x * blockDim.x)
        dst[i] = src[i];
}

// Copies a host block into the workspace through one of the context's pinned staging buffers
// (falls back to a pageable copy for blocks that do not fit).
int upload_block(cp_ctx* ctx, const std::vector<uint8_t>& block, void* dst, cudaStream_t s) {
    const size_t bytes = block.size();
    if (bytes > ctx->stage_bytes || (bytes & 15) != 0)
        return check_cuda(cudaMemcpyAsync(dst, block.data(), bytes, cudaMemcpyHostToDevice, s), "schedule copy");
    const int i = ctx->stage_next;
    ctx->stage_next = (i + 1) % kStageBuffers;
    if (ctx->stage_used[i])
        if (int rc = check_cuda(cudaEventSynchronize(ctx->stage_event[i]), "cudaEventSynchronize(stage)")) return rc;
    memcpy(ctx->h_stage[i], block.data(), bytes);
    const int64_t n16 = (int64_t)(bytes / 16);
    const int blocks = (int)std::min<int64_t>((n16 + 255) / 256, 64);
    stage_copy_kernel<<<blocks, 256, 0, s>>>(static_cast<uint4*>(dst), static_cast<const uint4*>(ctx->h_stage[i]), n16);
    if (int rc = check_cuda(cudaGetLastError(), "schedule copy launch")) return rc;
    ctx->stage_used[i] = true;
    return check_cuda(cudaEventRecord(ctx->stage_event[i], s), "cudaEventRecord(stage)");
}

// Page size for sizing a page table before the cache has been validated (a bad value is rejected later).
inline int64_t page_tokens_of(const cp_kv_cache* c) { return (c && c->page_size > 0) ? c->page_size : kDefaultPageTokens; }

int launch_fill_rows(float* out, float* lse, int64_t lse_stride, int64_t b, int64_t n, int32_t Hq, cudaStream_t s) {
    if (n <= 0) return CP_OK;
    const int64_t n4 = n * Hq * (kD / 4);
    fill_rows_kernel<<<(int)std::min<int64_t>((n4 + 255) / 256, 2048), 256, 0, s>>>(out, lse, lse_stride, b, n, Hq);
    return check_cuda(cudaGetLastError(), "fill_rows launch");
}

// want_fill: the call produces a partial result (fp32 out); rows it computes nothing for are written as zeros with
// lse = -inf (the identity element of cp_merge), by the attention kernel's spare warp.
int attn_common(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table, int32_t B,
                const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C, const int64_t* cu_pages,
                int32_t only_shard, int32_t only_chunk, int64_t kv_lo, int64_t kv_hi, int32_t Hq, float scale, void* out,
                int out_f32, bool want_fill, float* lse, void* workspace, size_t workspace_bytes, void* stream,
                const char* who, const cp_kv_cache_fp8* cache8 = nullptr) {
    if (!ctx || !q || !page_table || !out || !lse || B < 1 || !cu_new || !prefix_len || !C || !cu_pages)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer or B < 1", who);
    cp_kv_cache shape8;         // FP8 variant: the cache's shape in the bf16 descriptor's fields, for the shared logic
    if (cache8) {
        if (int rc = validate_kv_cache_fp8(cache8, who)) return rc;
        shape8.k = cache8->k;
        shape8.v = cache8->v;
        shape8.num_pages = cache8->num_pages;
        shape8.page_size = cache8->page_size;
        shape8.Hkv = cache8->Hkv;
        shape8.D = cache8->D;
        shape8.reserved = 0;
        shape8.stride_page = cache8->stride_page;
        shape8.stride_tok = cache8->stride_tok;
        shape8.stride_head = cache8->stride_head;
        cache = &shape8;
    } else if (int rc = validate_kv_cache(cache, who)) return rc;
    if (Hq < 1 || Hq % cache->Hkv != 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: Hq=%d is not a multiple of Hkv=%d", who, Hq, cache->Hkv);
    // even group size: two query heads of one KV group share every K/V tile; odd: one head per unit
    const int32_t heads_per_unit = ((Hq / cache->Hkv) % 2 == 0) ? 2 : 1;
    if (!(scale > 0.f)) return set_error(CP_ERR_INVALID_ARG, "%s: scale must be positive", who);
    if (((uintptr_t)q | (uintptr_t)out) & 15) return set_error(CP_ERR_INVALID_ARG, "%s: q and out must be 16-byte aligned", who);
    if (cu_new[0] != 0 || cu_pages[0] != 0) return set_error(CP_ERR_INVALID_ARG, "%s: cu_new[0] and cu_pages[0] must be 0", who);
    std::vector<int64_t> new_len(B);
    for (int32_t b = 0; b < B; ++b) {
        new_len[b] = cu_new[b + 1] - cu_new[b];
        if (new_len[b] < 1 || prefix_len[b] < 0 || C[b] < 1)
            return set_error(CP_ERR_INVALID_ARG, "%s: request %d has new_len=%lld prefix_len=%lld C=%d", who, b,
                             (long long)new_len[b], (long long)prefix_len[b], C[b]);
        const int64_t need = (prefix_len[b] + new_len[b] + cache->page_size - 1) / cache->page_size;
        if (cu_pages[b + 1] - cu_pages[b] < need)
            return set_error(CP_ERR_BOUNDS, "%s: request %d needs %lld page-table entries, has %lld", who, b,
                             (long long)need, (long long)(cu_pages[b + 1] - cu_pages[b]));
        if (prefix_len[b] + new_len[b] > 0x7fffff00ll)
            return set_error(CP_ERR_UNSUPPORTED, "%s: request %d is longer than 2^31 tokens", who, b);
    }
    if (cu_new[B] > 0x7fffff00ll || cu_pages[B] > 0x7fffff00ll)
        return set_error(CP_ERR_UNSUPPORTED, "%s: more than 2^31 packed rows or pages", who);
    const size_t base_ws = cp_workspace_bytes(B, new_len.data(), C, Hq);   // sized for one head per unit
    // FP8 variant: the quantised queries [rows, Hq, 128] and their scales [rows, Hq] follow the schedule space
    const size_t need_ws = cache8 ? cp_workspace_bytes_fp8(B, new_len.data(), C, Hq) : base_ws;
    if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need_ws)
        return set_error(CP_ERR_WORKSPACE, "%s: workspace %p of %zu bytes; need %zu bytes, 256-byte aligned", who,
                         workspace, workspace_bytes, need_ws);

    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int grid_max = ctx->num_sms;
    uint8_t* ws = static_cast<uint8_t*>(workspace);
    // With schedule reuse on, a call whose schedule-relevant arguments and workspace equal the previous call's
    // (the next layer of the same batch) launches on the work lists that are already in the workspace.
    std::vector<int64_t> key;
    if (ctx->cache_on) {
        key.reserve(14 + 4 * (size_t)B);
        const int64_t head[] = {B, Hq, cache->Hkv, cache->page_size, only_shard, only_chunk, kv_lo, kv_hi,
                                grid_max, out_f32, want_fill, cache8 != nullptr};
        key.assign(head, head + sizeof head / sizeof head[0]);
        for (int32_t b = 0; b < B; ++b) {
            key.push_back(cu_new[b + 1]); key.push_back(prefix_len[b]); key.push_back(C[b]); key.push_back(cu_pages[b + 1]);
        }
    }
    WorkspaceLayout lay;        // where the partial results (and the lists of a large schedule) sit in the workspace
    WorkspaceLayout ilay;       // offsets of the lists inside the launch-parameter copy of a small schedule
    int32_t grid, n_items, n_merges, n_fill = 0;
    int32_t fill[2 * kMaxFillRanges] = {0};
    int64_t total_rows;
    bool inl_on = false;
    bool fill_all = false;      // more uncovered row ranges than the kernel takes: a fill launch precedes the attention launch
    InlineSched inl_local;
    inl_local.bytes[0] = 0;
    const InlineSched* inl = &inl_local;
    if (ctx->cache_on && ctx->cache_valid && ctx->cache_ws == workspace && ctx->cache_args == key) {
        lay = ctx->cache_lay;
        grid = ctx->cache_grid;
        n_items = ctx->cache_items;
        n_merges = ctx->cache_merges;
        total_rows = ctx->cache_rows;
        inl_on = ctx->cache_inline;
        inl = &ctx->cache_inl;
        n_fill = ctx->cache_n_fill;
        memcpy(fill, ctx->cache_fill, sizeof fill);
        fill_all = ctx->cache_fill_all;
    } else {
        ctx->cache_valid = false;
        Schedule sch;
        // even groups: 128-row tiles for pairs of heads; odd groups: 256-row tile pairs for single heads
        build_tiles(B, cu_new, prefix_len, C, cu_pages, cache->page_size, only_shard, only_chunk, kv_lo, kv_hi,
                    heads_per_unit == 2 ? kTileRows : 2 * kTileRows, sch.items);
        // rows of q / out / lse: the packed batch, or the one chunk of a chunk call
        total_rows = cu_new[B];
        if (only_chunk >= 0) {
            total_rows = 0;
            for (const TileItem& t : sch.items) total_rows = std::max<int64_t>(total_rows, (int64_t)t.q_row0 + t.n_rows);
        }
        if (sch.items.empty())   // the shard owns no rows (only empty chunks), or no row sees a key of the range
            return want_fill ? launch_fill_rows(static_cast<float*>(out), lse, total_rows, 0, total_rows, Hq, s) : CP_OK;
        if (want_fill) {
            int64_t gaps[2 * kMaxFillRanges];
            const int n = uncovered_rows(sch.items, total_rows, gaps, kMaxFillRanges);
            if (n > kMaxFillRanges) {     // more gaps than the kernel takes: fill everything first, in stream order
                fill_all = true;
            } else {
                n_fill = n;
                for (int i = 0; i < 2 * n; ++i) fill[i] = (int32_t)gaps[i];
            }
        }
        if (int rc = build_schedule(Hq / heads_per_unit,
                                    kv_major_pairs(B, cu_new, prefix_len, cache->Hkv, (Hq / cache->Hkv) / heads_per_unit),
                                    grid_max, sch)) return rc;
        if (n_fill > 0 && sch.grid < std::min(grid_max, kMaxGrid)) {
            // rows to fill: CTAs without work join the launch so that every SM's spare warp shares the stores
            sch.grid = std::min(grid_max, kMaxGrid);
            sch.cta_off.resize((size_t)sch.grid + 1, sch.cta_off.back());
        }
        lay = workspace_layout(sch.items.size(), sch.pieces.size(), sch.merges.size(), sch.merge_slots.size(), sch.grid,
                               sch.n_slots);
        if (lay.total > workspace_bytes)
            return set_error(CP_ERR_WORKSPACE, "%s: schedule needs %zu workspace bytes, have %zu", who, lay.total, workspace_bytes);
        // one contiguous block: items | cta_off | pieces | merges | merge_slots.  A block of at most
        // kInlineSchedBytes (packed to 16-byte boundaries) rides in the launch parameters; a larger one is copied
        // into the workspace by a small kernel.
        ilay = workspace_layout(sch.items.size(), sch.pieces.size(), sch.merges.size(), sch.merge_slots.size(), sch.grid,
                                0, 16);
        inl_on = ilay.partial_o - ilay.items <= kInlineSchedBytes;
        const WorkspaceLayout& bl = inl_on ? ilay : lay;
        std::vector<uint8_t> big;
        uint8_t* block = inl_local.bytes;
        if (!inl_on) {
            big.assign(bl.partial_o - bl.items, 0);
            block = big.data();
        }
        memcpy(block + (bl.items - bl.items), sch.items.data(), sch.items.size() * sizeof(TileItem));
        memcpy(block + (bl.cta_off - bl.items), sch.cta_off.data(), sch.cta_off.size() * sizeof(int32_t));
        memcpy(block + (bl.pieces - bl.items), sch.pieces.data(), sch.pieces.size() * sizeof(PieceEntry));
        if (!sch.merges.empty()) {
            memcpy(block + (bl.merges - bl.items), sch.merges.data(), sch.merges.size() * sizeof(MergeEntry));
            memcpy(block + (bl.merge_slots - bl.items), sch.merge_slots.data(), sch.merge_slots.size() * sizeof(int32_t));
        }
        if (inl_on) {
            // the list offsets inside the parameter block take the place of the workspace offsets
            const size_t base = ilay.items;
            lay.items = ilay.items - base;
            lay.cta_off = ilay.cta_off - base;
            lay.pieces = ilay.pieces - base;
            lay.merges = ilay.merges - base;
            lay.merge_slots = ilay.merge_slots - base;
        } else {
            // the staged upload reads a pinned buffer that later calls reuse: a captured copy would replay stale lists
            cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
            if (int rc = check_cuda(cudaStreamIsCapturing(s, &cap), "cudaStreamIsCapturing")) return rc;
            if (cap != cudaStreamCaptureStatusNone)
                return set_error(CP_ERR_UNSUPPORTED, "%s: the work lists (%zu bytes) do not fit the launch parameters (%zu); "
                                 "a call of this size cannot be captured into a CUDA graph", who, big.size(), kInlineSchedBytes);
            if (int rc = upload_block(ctx, big, ws + lay.items, s)) return rc;
        }
        grid = sch.grid;
        n_items = (int32_t)sch.items.size();
        n_merges = (int32_t)sch.merges.size();
        if (ctx->cache_on) {
            ctx->cache_valid = true;
            ctx->cache_args = std::move(key);
            ctx->cache_ws = workspace;
            ctx->cache_lay = lay;
            ctx->cache_grid = grid;
            ctx->cache_items = n_items;
            ctx->cache_merges = n_merges;
            ctx->cache_rows = total_rows;
            ctx->cache_inline = inl_on;
            if (inl_on) memcpy(ctx->cache_inl.bytes, inl_local.bytes, kInlineSchedBytes);
            ctx->cache_n_fill = n_fill;
            memcpy(ctx->cache_fill, fill, sizeof fill);
            ctx->cache_fill_all = fill_all;
        }
    }

    if (fill_all)
        if (int rc = launch_fill_rows(static_cast<float*>(out), lse, total_rows, 0, total_rows, Hq, s)) return rc;
    CUtensorMap tmQ, tmK, tmV;
    uint8_t* q8 = ws + base_ws;
    float* q_scale = reinterpret_cast<float*>(q8 + (size_t)total_rows * Hq * kD);
    if (cache8) {
        // quantise the queries once per call (a unit cut along KV would otherwise repeat it per piece)
        const int64_t n_rows = total_rows * Hq;
        quantize_q_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, s>>>(static_cast<const __nv_bfloat16*>(q), q8, q_scale, n_rows);
        if (int rc = check_cuda(cudaGetLastError(), "quantize_q launch")) return rc;
    }
    // a tensor map depends only on addresses, shapes and strides: the previous call's maps serve again when
    // those are unchanged (encoding three maps costs a few microseconds of host time)
    const int64_t mkey[12] = {(int64_t)(uintptr_t)(cache8 ? (const void*)q8 : q), total_rows, Hq, cache8 ? 1 : 0,
                              (int64_t)(uintptr_t)cache->k, (int64_t)(uintptr_t)cache->v, cache->num_pages, cache->page_size,
                              cache->Hkv, cache->stride_page, cache->stride_tok, cache->stride_head};
    if (ctx->maps_valid && memcmp(mkey, ctx->maps_key, sizeof mkey) == 0) {
        tmQ = ctx->maps[0];
        tmK = ctx->maps[1];
        tmV = ctx->maps[2];
    } else {
        if (cache8) {
            if (int rc = encode_maps_fp8(ctx, q8, total_rows, Hq, cache8, &tmQ, &tmK, &tmV)) return rc;
        } else if (int rc = encode_maps(ctx, q, total_rows, Hq, cache, &tmQ, &tmK, &tmV)) {
            return rc;
        }
        memcpy(ctx->maps_key, mkey, sizeof mkey);
        ctx->maps[0] = tmQ;
        ctx->maps[1] = tmK;
        ctx->maps[2] = tmV;
        ctx->maps_valid = true;
    }
    if (!ctx->attn_attr_set) {
        if (int rc = check_cuda(cudaFuncSetAttribute(cp_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)kSmemAlloc), "cudaFuncSetAttribute(attn)")) return rc;
        if (int rc = check_cuda(cudaFuncSetAttribute(cp_attn_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)kSmemAlloc), "cudaFuncSetAttribute(attn)")) return rc;
        ctx->attn_attr_set = true;
    }
    AttnParams p;
    p.items = reinterpret_cast<const TileItem*>(ws + lay.items);
    p.n_items = n_items;
    p.cta_off = reinterpret_cast<const int32_t*>(ws + lay.cta_off);
    p.pieces = reinterpret_cast<const PieceEntry*>(ws + lay.pieces);
    p.inl_items = p.inl_cta_off = p.inl_pieces = -1;
    if (inl_on) {
        p.items = nullptr;
        p.cta_off = nullptr;
        p.pieces = nullptr;
        p.inl_items = (int32_t)lay.items;
        p.inl_cta_off = (int32_t)lay.cta_off;
        p.inl_pieces = (int32_t)lay.pieces;
    }
    p.partial_o = reinterpret_cast<float*>(ws + lay.partial_o);
    p.partial_lse = reinterpret_cast<float*>(ws + lay.partial_lse);
    p.pairs_per_tile = Hq / heads_per_unit;
    p.pairs_per_kv = 0;
    p.heads_per_unit = heads_per_unit;
    p.group = Hq / cache->Hkv;
    p.Hq = Hq;
    p.page_table = page_table;
    p.oob_page = (int32_t)std::min<int64_t>(cache->num_pages, 0x7fffffff);
    p.page_tokens = cache->page_size;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.out = out;
    p.out_f32 = out_f32;
    p.lse = lse;
    p.lse_stride = total_rows;
    p.status = ctx->d_status;
    p.n_fill = n_fill;
    memcpy(p.fill, fill, sizeof fill);
    p.q_scale = cache8 ? q_scale : nullptr;
    p.k_scale = cache8 ? cache8->k_scale : nullptr;
    p.v_scale = cache8 ? cache8->v_scale : nullptr;
    p.co_producer = (!cache8 && cache->page_size == 16 && n_fill == 0) ? 1 : 0;
    if (cache8) cp_attn_kernel<true><<<grid, kThreads, kSmemAlloc, s>>>(tmQ, tmK, tmV, p, *inl);
    else cp_attn_kernel<false><<<grid, kThreads, kSmemAlloc, s>>>(tmQ, tmK, tmV, p, *inl);
    if (int rc = check_cuda(cudaGetLastError(), who)) return rc;
    if (n_merges > 0) {
        FixupParams f;
        f.items = p.items;
        f.merges = reinterpret_cast<const MergeEntry*>(ws + lay.merges);
        f.merge_slots = reinterpret_cast<const int32_t*>(ws + lay.merge_slots);
        f.inl_items = f.inl_merges = f.inl_merge_slots = -1;
        if (inl_on) {
            f.merges = nullptr;
            f.merge_slots = nullptr;
            f.inl_items = (int32_t)lay.items;
            f.inl_merges = (int32_t)lay.merges;
            f.inl_merge_slots = (int32_t)lay.merge_slots;
        }
        f.partial_o = p.partial_o;
        f.partial_lse = p.partial_lse;
        f.out = out;
        f.out_f32 = out_f32;
        f.Hq = Hq;
        f.heads_per_unit = heads_per_unit;
        f.lse = lse;
        f.lse_stride = total_rows;
        cp_attn_fixup_kernel<<<dim3((unsigned)n_merges, 2 * kBlockM / kFixupRowsPerBlock), 256, 0, s>>>(f, *inl);
        if (int rc = check_cuda(cudaGetLastError(), "cp_attn_fixup launch")) return rc;
    }
    return CP_OK;
}

}  // namespace

extern "C" int cp_prefill_attn_batch(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                                     int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                                     const int64_t* cu_pages, int32_t Hq, float scale, void* out, float* lse,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    return attn_common(ctx, q, cache, page_table, B, cu_new, prefix_len, C, cu_pages, -1, -1, 0, INT32_MAX, Hq, scale, out, 0,
                       false, lse, workspace, workspace_bytes, stream, "cp_prefill_attn_batch");
}

extern "C" int cp_prefill_attn(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                               int64_t prefix_len, int64_t new_len, int32_t C, int32_t Hq, float scale, void* out,
                               float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!cache || new_len < 1 || prefix_len < 0)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn: cache is NULL, new_len < 1 or prefix_len < 0");
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + page_tokens_of(cache) - 1) / page_tokens_of(cache)};
    return attn_common(ctx, q, cache, page_table, 1, cu_new, &prefix_len, &C, cu_pages, -1, -1, 0, INT32_MAX, Hq, scale, out, 0,
                       false, lse, workspace, workspace_bytes, stream, "cp_prefill_attn");
}

extern "C" int cp_prefill_attn_fp8_batch(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                                         int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                                         const int64_t* cu_pages, int32_t Hq, float scale, void* out, float* lse,
                                         void* workspace, size_t workspace_bytes, void* stream) {
    if (!cache) return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_fp8_batch: cache is NULL");
    return attn_common(ctx, q, nullptr, page_table, B, cu_new, prefix_len, C, cu_pages, -1, -1, 0, INT32_MAX, Hq, scale, out, 0,
                       false, lse, workspace, workspace_bytes, stream, "cp_prefill_attn_fp8_batch", cache);
}

extern "C" int cp_prefill_attn_fp8(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                                   int64_t prefix_len, int64_t new_len, int32_t C, int32_t Hq, float scale, void* out,
                                   float* lse, void* workspace, size_t workspace_bytes, void* stream) {
    if (!cache || new_len < 1 || prefix_len < 0 || cache->page_size < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_fp8: cache is NULL, new_len < 1 or prefix_len < 0");
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + cache->page_size - 1) / cache->page_size};
    return attn_common(ctx, q, nullptr, page_table, 1, cu_new, &prefix_len, &C, cu_pages, -1, -1, 0, INT32_MAX, Hq, scale, out, 0,
                       false, lse, workspace, workspace_bytes, stream, "cp_prefill_attn_fp8", cache);
}

// The one-shard, one-chunk and key-range calls of the FP8 variant: the same tile lists as their bf16 forms.
extern "C" int cp_prefill_attn_fp8_shard(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                                         int64_t prefix_len, int64_t new_len, int32_t C, int32_t shard, int32_t Hq,
                                         float scale, float* partial_out, float* partial_lse, void* workspace,
                                         size_t workspace_bytes, void* stream) {
    if (!cache || cache->page_size < 1 || new_len < 1 || prefix_len < 0 || C < 1 || shard < 0 || shard >= C || !partial_out ||
        !partial_lse || Hq < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_fp8_shard: bad sizes or shard %d not in [0, %d)", shard, C);
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + cache->page_size - 1) / cache->page_size};
    return attn_common(ctx, q, nullptr, page_table, 1, cu_new, &prefix_len, &C, cu_pages, shard, -1, 0, INT32_MAX, Hq, scale,
                       partial_out, 1, true, partial_lse, workspace, workspace_bytes, stream, "cp_prefill_attn_fp8_shard", cache);
}

extern "C" int cp_prefill_attn_fp8_chunk(cp_ctx* ctx, const void* q_chunk, const cp_kv_cache_fp8* cache,
                                         const int32_t* page_table, int64_t prefix_len, int64_t new_len, int32_t C,
                                         int32_t chunk, int32_t Hq, float scale, void* out_chunk, float* lse_chunk,
                                         void* workspace, size_t workspace_bytes, void* stream) {
    if (!cache || cache->page_size < 1 || new_len < 1 || prefix_len < 0 || C < 1 || chunk < 0 || chunk >= 2 * (int64_t)C)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_fp8_chunk: bad sizes or chunk %d not in [0, %d)", chunk, 2 * C);
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + cache->page_size - 1) / cache->page_size};
    return attn_common(ctx, q_chunk, nullptr, page_table, 1, cu_new, &prefix_len, &C, cu_pages, -1, chunk, 0, INT32_MAX, Hq,
                       scale, out_chunk, 0, false, lse_chunk, workspace, workspace_bytes, stream, "cp_prefill_attn_fp8_chunk",
                       cache);
}

extern "C" int cp_prefill_attn_fp8_kvrange(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                                           int64_t prefix_len, int64_t new_len, int64_t kv_lo, int64_t kv_hi, int32_t Hq,
                                           float scale, float* partial_out, float* partial_lse, void* workspace,
                                           size_t workspace_bytes, void* stream) {
    if (!cache || cache->page_size < 1 || new_len < 1 || prefix_len < 0 || !partial_out || !partial_lse || Hq < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_fp8_kvrange: null pointer or bad sizes");
    if (kv_lo < 0 || kv_hi < kv_lo || kv_lo > 0x7fffff00ll)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_fp8_kvrange: key range [%lld, %lld)", (long long)kv_lo, (long long)kv_hi);
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + cache->page_size - 1) / cache->page_size};
    const int32_t C = 1;
    return attn_common(ctx, q, nullptr, page_table, 1, cu_new, &prefix_len, &C, cu_pages, -1, -1, kv_lo,
                       std::min<int64_t>(kv_hi, INT32_MAX), Hq, scale, partial_out, 1, true, partial_lse, workspace,
                       workspace_bytes, stream, "cp_prefill_attn_fp8_kvrange", cache);
}

// The two partial-result calls write zeros with lse = -inf (the identity element of cp_merge) into the rows
// they compute nothing for; the attention kernel's spare warp does it, so each call is one launch.
extern "C" int cp_prefill_attn_shard(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                                     int64_t prefix_len, int64_t new_len, int32_t C, int32_t shard, int32_t Hq,
                                     float scale, float* partial_out, float* partial_lse, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    if (!cache || new_len < 1 || prefix_len < 0 || C < 1 || shard < 0 || shard >= C || !partial_out || !partial_lse || Hq < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_shard: bad sizes or shard %d not in [0, %d)", shard, C);
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + page_tokens_of(cache) - 1) / page_tokens_of(cache)};
    return attn_common(ctx, q, cache, page_table, 1, cu_new, &prefix_len, &C, cu_pages, shard, -1, 0, INT32_MAX, Hq, scale,
                       partial_out, 1, true, partial_lse, workspace, workspace_bytes, stream, "cp_prefill_attn_shard");
}

extern "C" int cp_prefill_attn_kvrange(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                                       int64_t prefix_len, int64_t new_len, int64_t kv_lo, int64_t kv_hi, int32_t Hq,
                                       float scale, float* partial_out, float* partial_lse, void* workspace,
                                       size_t workspace_bytes, void* stream) {
    if (!cache || new_len < 1 || prefix_len < 0 || !partial_out || !partial_lse || Hq < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_kvrange: null pointer or bad sizes");
    if (kv_lo < 0 || kv_hi < kv_lo || kv_lo > 0x7fffff00ll)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_kvrange: key range [%lld, %lld)", (long long)kv_lo, (long long)kv_hi);
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + page_tokens_of(cache) - 1) / page_tokens_of(cache)};
    const int32_t C = 1;
    return attn_common(ctx, q, cache, page_table, 1, cu_new, &prefix_len, &C, cu_pages, -1, -1, kv_lo,
                       std::min<int64_t>(kv_hi, INT32_MAX), Hq, scale, partial_out, 1, true, partial_lse, workspace,
                       workspace_bytes, stream, "cp_prefill_attn_kvrange");
}

extern "C" int cp_ctx_selftest_wait_expiry(cp_ctx* ctx, void* stream) {
    if (!ctx) return set_error(CP_ERR_INVALID_ARG, "cp_ctx_selftest_wait_expiry: ctx is NULL");
    if (int rc = check_cuda(cudaSetDevice(ctx->device), "cudaSetDevice")) return rc;
    wait_expiry_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_status, 2000000ll);
    return check_cuda(cudaGetLastError(), "cp_ctx_selftest_wait_expiry launch");
}

extern "C" int cp_prefill_attn_chunk(cp_ctx* ctx, const void* q_chunk, const cp_kv_cache* cache, const int32_t* page_table,
                                     int64_t prefix_len, int64_t new_len, int32_t C, int32_t chunk, int32_t Hq,
                                     float scale, void* out_chunk, float* lse_chunk, void* workspace,
                                     size_t workspace_bytes, void* stream) {
    if (!cache || new_len < 1 || prefix_len < 0 || C < 1 || chunk < 0 || chunk >= 2 * (int64_t)C)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefill_attn_chunk: bad sizes or chunk %d not in [0, %d)", chunk, 2 * C);
    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + page_tokens_of(cache) - 1) / page_tokens_of(cache)};
    return attn_common(ctx, q_chunk, cache, page_table, 1, cu_new, &prefix_len, &C, cu_pages, -1, chunk, 0, INT32_MAX, Hq,
                       scale, out_chunk, 0, false, lse_chunk, workspace, workspace_bytes, stream, "cp_prefill_attn_chunk");
}

// ------------------------------------------------------------------------------------------------
// cp_prefill_attn_static: the single-request call for callers that may not allocate.
// The tile list and the status words live in a fixed device array that is part of the library
// image; nothing here calls an allocating CUDA routine and no cp_ctx is needed.
// ------------------------------------------------------------------------------------------------
namespace {

constexpr int kStaticMaxTiles = 2048;   // 128-row query tiles: 262,144 new tokens
constexpr size_t kStaticScratchBytes = kWorkspaceHeader + (size_t)kStaticMaxTiles * sizeof(TileItem);
constexpr int kStaticMaxDevices = 64;

// [0, 16): status words {code, barrier, block, iteration}; [256, ...): tile list.
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct StaticDeviceState {
    bool ready;
    unsigned char* scratch;     // device address of g_static_scratch on this device
    int num_sms;
    EncodeTiledFn encode_tiled;
};
StaticDeviceState g_static_state[kStaticMaxDevices];

// One-time set-up for the current device: resolve the device address of the scratch array (its name
// in host code is only a handle), the tensor-map encoder and the kernel's shared-memory limit.
int static_setup(int device, StaticDeviceState** out) {
    if (device < 0 || device >= kStaticMaxDevices)
        return set_error(CP_ERR_UNSUPPORTED, "cp_prefill_attn_static: device ordinal %d not supported", device);
    StaticDeviceState& st = g_static_state[device];
    if (!st.ready) {
        void* ptr = nullptr;
        if (int rc = check_cuda(cudaGetSymbolAddress(&ptr, g_static_scratch), "cudaGetSymbolAddress(static scratch)"))
            return rc;
        cudaDeviceProp prop;
        if (int rc = check_cuda(cudaGetDeviceProperties(&prop, device), "cudaGetDeviceProperties")) return rc;
        if (prop.major != 10)
            return set_error(CP_ERR_UNSUPPORTED, "cp_prefill_attn_static: device is sm_%d%d, sm_100a only", prop.major, prop.minor);
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (int rc = check_cuda(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q),
                                "cudaGetDriverEntryPoint(cuTensorMapEncodeTiled)")) return rc;
        if (q != cudaDriverEntryPointSuccess || !fn)
            return set_error(CP_ERR_CUDA, "cuTensorMapEncodeTiled is not available in this driver");
        if (int rc = check_cuda(cudaFuncSetAttribute(cp_attn_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                     (int)kSmemAlloc), "cudaFuncSetAttribute(attn)")) return rc;
        st.scratch = static_cast<unsigned char*>(ptr);
        st.num_sms = prop.multiProcessorCount;
        st.encode_tiled = reinterpret_cast<EncodeTiledFn>(fn);
        st.ready = true;
    }
    *out = &st;
    return CP_OK;
}

// Writes the request's tile list into the scratch and clears the status words, from the lengths alone (the
// all-shards tile list is plain arithmetic: tile t covers rows [128 t, 128 t + 128), longest tiles first), so no
// host buffer is read when the stream runs.
__global__ void static_tiles_kernel(unsigned char* scratch, int64_t R, int64_t P, int32_t n_pages, int32_t n_tiles,
                                    int32_t tile_rows) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < kStatusWords) reinterpret_cast<int32_t*>(scratch)[i] = 0;
    if (i >= n_tiles) return;
    const int64_t r0 = (int64_t)(n_tiles - 1 - i) * tile_rows;
    TileItem t;
    t.q_row0 = (int32_t)r0;
    t.n_rows = (int32_t)min((int64_t)tile_rows, R - r0);
    t.kv_len0 = (int32_t)(P + r0 + 1);
    t.pt_base = 0;
    t.n_pages = n_pages;
    t.n_kv_tiles = (int32_t)((P + r0 + t.n_rows + kTileRows - 1) / kTileRows);
    t.kv_lo = 0;
    t.kv_hi = INT32_MAX;
    reinterpret_cast<TileItem*>(scratch + kWorkspaceHeader)[i] = t;
}

}  // namespace

extern "C" int cp_prefill_attn_static(const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                                      int64_t prefix_len, int64_t new_len, int32_t C, int32_t Hq, float scale,
                                      void* out, float* lse, void* stream) {
    const char* who = "cp_prefill_attn_static";
    if (!q || !page_table || !out || !lse || new_len < 1 || prefix_len < 0 || C < 1)
        return set_error(CP_ERR_INVALID_ARG, "%s: null pointer, new_len < 1, prefix_len < 0 or C < 1", who);
    if (int rc = validate_kv_cache(cache, who)) return rc;
    if (Hq < 1 || Hq % cache->Hkv != 0)
        return set_error(CP_ERR_INVALID_ARG, "%s: Hq=%d is not a multiple of Hkv=%d", who, Hq, cache->Hkv);
    const int32_t heads_per_unit = ((Hq / cache->Hkv) % 2 == 0) ? 2 : 1;
    if (!(scale > 0.f)) return set_error(CP_ERR_INVALID_ARG, "%s: scale must be positive", who);
    if (((uintptr_t)q | (uintptr_t)out) & 15) return set_error(CP_ERR_INVALID_ARG, "%s: q and out must be 16-byte aligned", who);
    if (prefix_len + new_len > 0x7fffff00ll) return set_error(CP_ERR_UNSUPPORTED, "%s: request longer than 2^31 tokens", who);
    const int32_t tile_rows = heads_per_unit == 2 ? kTileRows : 2 * kTileRows;      // single-head units take tile pairs
    const int64_t n_tiles = (new_len + tile_rows - 1) / tile_rows;
    if ((new_len + kTileRows - 1) / kTileRows > kStaticMaxTiles)
        return set_error(CP_ERR_WORKSPACE, "%s: new_len=%lld needs %lld query tiles; the built-in scratch holds %d "
                         "(use cp_prefill_attn with a caller workspace)", who, (long long)new_len,
                         (long long)((new_len + kTileRows - 1) / kTileRows), kStaticMaxTiles);
    int device = -1;
    if (int rc = check_cuda(cudaGetDevice(&device), "cudaGetDevice")) return rc;
    StaticDeviceState* st = nullptr;
    if (int rc = static_setup(device, &st)) return rc;

    const int64_t cu_new[2] = {0, new_len};
    const int64_t cu_pages[2] = {0, (prefix_len + new_len + page_tokens_of(cache) - 1) / page_tokens_of(cache)};
    cp_ctx enc{};                       // only the encoder entry point is read by encode_maps
    enc.encode_tiled = st->encode_tiled;
    CUtensorMap tmQ, tmK, tmV;
    if (int rc = encode_maps(&enc, q, new_len, Hq, cache, &tmQ, &tmK, &tmV)) return rc;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // The scratch keeps whatever the previous call left: a small kernel clears the status words and writes this
    // request's tile list in stream order (no host memory is read later, whatever the stream does with the work).
    static_tiles_kernel<<<(unsigned)((n_tiles + 255) / 256), 256, 0, s>>>(
        st->scratch, new_len, prefix_len, (int32_t)cu_pages[1], (int32_t)n_tiles, tile_rows);
    if (int rc = check_cuda(cudaGetLastError(), "static tile list launch")) return rc;
    AttnParams p;
    p.items = reinterpret_cast<const TileItem*>(st->scratch + kWorkspaceHeader);
    p.n_items = (int32_t)n_tiles;
    p.cta_off = nullptr;       // implicit schedule over whole units: no piece lists, no partial results
    p.pieces = nullptr;
    p.partial_o = nullptr;
    p.partial_lse = nullptr;
    p.pairs_per_tile = Hq / heads_per_unit;
    p.pairs_per_kv = kv_major_pairs(1, cu_new, &prefix_len, cache->Hkv, (Hq / cache->Hkv) / heads_per_unit);
    p.heads_per_unit = heads_per_unit;
    p.group = Hq / cache->Hkv;
    p.Hq = Hq;
    p.page_table = page_table;
    p.oob_page = (int32_t)std::min<int64_t>(cache->num_pages, 0x7fffffff);
    p.page_tokens = cache->page_size;
    p.scale_log2 = scale * 1.4426950408889634f;
    p.out = out;
    p.out_f32 = 0;
    p.lse = lse;
    p.lse_stride = new_len;
    p.status = reinterpret_cast<int32_t*>(st->scratch);
    p.inl_items = p.inl_cta_off = p.inl_pieces = -1;
    p.n_fill = 0;
    p.q_scale = p.k_scale = p.v_scale = nullptr;
    p.co_producer = cache->page_size == 16 ? 1 : 0;
    InlineSched none;          // unused: the tile list is in the scratch
    none.bytes[0] = 0;
    const int64_t units = n_tiles * p.pairs_per_tile;
    const int grid = (int)std::min<int64_t>(units, st->num_sms);
    cp_attn_kernel<false><<<grid, kThreads, kSmemAlloc, s>>>(tmQ, tmK, tmV, p, none);
    return check_cuda(cudaGetLastError(), who);
}

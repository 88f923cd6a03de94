/*
 * libcpattn -- cache-aware causal prefill attention under zigzag context parallelism (CP),
 * hand-written for NVIDIA B200 (sm_100a).  C ABI.
 *
 * Notation (paper Sections 2.1-2.2): P = prefix_len, the cached tokens of a request;
 * R = new_len, its uncached suffix (the only tokens that are queries); L = P + R; C = CP
 * degree; Hq / Hkv query / KV heads, G = Hq / Hkv; D = head dimension.  New token r sits at
 * absolute position P + r and attends to keys 0 .. P + r (diagonal included).
 *
 * Conventions
 *   - Every call returns an int: CP_OK (0) or a negative CP_ERR_* code; cp_strerror() names the
 *     code and cp_last_error() gives a per-thread message for the last failing call.
 *   - All buffers are owned by the caller.  "device" pointers are CUDA device memory of the
 *     context's device, "host" pointers ordinary host memory.  The library allocates device
 *     memory only inside cp_ctx_create().
 *   - GPU calls validate their arguments first (an invalid call launches nothing), then only
 *     ENQUEUE work on the given stream (a cudaStream_t passed as void*, NULL = default stream)
 *     and return.  Device-side failures (a bounded wait that ran out, a page id outside the pool
 *     met by a paged copy) are recorded in a status word that cp_ctx_poll_status() reads after the
 *     caller has synchronised.
 *   - bf16 tensors are passed as void*; element strides are in elements.
 *   - Stream capture: an attention call with a cp_ctx whose work lists ride in the launch parameters
 *     (cp_schedule_inspect reports it; up to 24 KB of lists, i.e. a few hundred work units) reads no host
 *     memory after it returns and may be captured into a CUDA graph and replayed; a call with a larger
 *     schedule stages its lists through the context's pinned buffers, which later calls reuse: such a
 *     call on a capturing stream returns CP_ERR_UNSUPPORTED and enqueues nothing.  cp_merge and the paged copies take everything by value and may be captured.
 */
#ifndef CPATTN_H
#define CPATTN_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    CP_OK = 0,
    CP_ERR_INVALID_ARG = -1, /* null pointer, non-positive size, inconsistent lengths              */
    CP_ERR_UNSUPPORTED = -2, /* D != 128, unsupported page size, misaligned strides, sizes beyond limits */
    CP_ERR_WORKSPACE = -3,   /* workspace missing, misaligned or smaller than cp_workspace_bytes() */
    CP_ERR_CUDA = -4,        /* a CUDA runtime / driver call failed                                */
    CP_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired (reported by poll_status)       */
    CP_ERR_BOUNDS = -6       /* an index is out of range: a page-table size seen by the host, or a
                                page id met by cp_kv_gather / cp_kv_append on the device (poll_status) */
};

enum { CP_DTYPE_BF16 = 0, CP_DTYPE_F32 = 1 };

const char* cp_strerror(int code);
const char* cp_last_error(void);

/* ---------------------------------------------------------------------------------------------
 * Context: one per (host thread, device).  Holds the device status word, the pinned staging
 * buffer for tile lists and the resolved driver entry point for tensor-map encoding.
 * cp_ctx_create() makes `device` current and allocates; cp_ctx_destroy() frees.
 * cp_ctx_poll_status() synchronises the device-to-host copy of the status word on the default
 * stream (call it after synchronising the streams you used): returns CP_OK, CP_ERR_TIMEOUT or
 * CP_ERR_BOUNDS and, when `detail` is non-NULL, writes 4 int32 words ({code, barrier id, block,
 * iteration} for a time-out, {code, page-table index, block, page id} for a bad page id); the
 * status word is cleared by the call.
 * ------------------------------------------------------------------------------------------- */
typedef struct cp_ctx cp_ctx;
int cp_ctx_create(cp_ctx** ctx, int device);
int cp_ctx_destroy(cp_ctx* ctx);
int cp_ctx_poll_status(cp_ctx* ctx, int32_t* detail /* host, 4 words or NULL */);

/* cp_ctx_cache_schedule -- schedule reuse, off by default.  The layers of a model call the attention entry
 * points with the same batch over and over (same lengths, C, head counts, page-table sizes; only q, the
 * cache contents and out differ).  With reuse on, a call whose schedule-relevant arguments AND workspace are
 * the previous call's skips the host-side scheduling and the upload and launches on the work lists already
 * in the workspace (about 20-100 us of host time per call and one small kernel).  While it is on, the caller
 * must not modify the workspace between such calls, nor hand it to another context, and must issue the
 * calls on one stream (or order the streams behind the first call: a large schedule is uploaded on the stream
 * of the call that built it).  Turning it on or off forgets the remembered schedule.  Errors: INVALID_ARG. */
int cp_ctx_cache_schedule(cp_ctx* ctx, int enable);

/* cp_ctx_selftest_wait_expiry -- diagnostic (the paper has no counterpart): enqueues one small block whose
 * only act is to wait, with a limit of about a millisecond, on a barrier that nothing arrives at.  It shows
 * on the device at hand that an expired wait ends the kernel normally and is reported: after the stream has
 * been synchronised, cp_ctx_poll_status returns CP_ERR_TIMEOUT with detail {code, barrier 0, block 0,
 * iteration 7} and clears the status; the context stays usable.  Errors: INVALID_ARG, CUDA. */
int cp_ctx_selftest_wait_expiry(cp_ctx* ctx, void* stream);

/* ---------------------------------------------------------------------------------------------
 * cp_plan -- zigzag shard plan (paper Section 2.1, applied to the uncached suffix of Section 2.2).
 * The R new tokens are padded on the right to a multiple of 2C: chunk length cl = ceil(R / 2C);
 * chunk j = [min(j*cl, R), min((j+1)*cl, R)) (trailing chunks may be short or empty); shard k owns
 * chunks k and 2C-1-k.  A chunk ending at q_end needs keys [0, P + q_end).  `pairs` is the number
 * of visible (query, key) pairs of the shard; over all shards it sums to W(R,P) = R*P + R(R+1)/2
 * (Eq. 1).  Host only, integer only.  out: host array of C entries.
 * Errors: CP_ERR_INVALID_ARG if new_len < 1, prefix_len < 0, C < 1 or out == NULL.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    int64_t q_begin[2]; /* new-token index, half-open; [0] = chunk k, [1] = chunk 2C-1-k */
    int64_t q_end[2];
    int64_t kv_end[2];  /* absolute, exclusive: P + q_end (kv_begin is always 0)          */
    uint64_t pairs;
} cp_shard_plan;
int cp_plan(int64_t new_len, int64_t prefix_len, int32_t C, cp_shard_plan* out);

/* ---------------------------------------------------------------------------------------------
 * Paged KV cache.  Logical token t of a request, KV head g, dim d lives at element
 *   page_table[t / page_size] * stride_page + (t % page_size) * stride_tok + g * stride_head + d.
 * The new tokens' K and V are already in the cache at logical positions [P, P+R) when attention is
 * called (the ranks gather K/V before attending, Section 2.1).  Default layout
 * [num_pages, 64, Hkv, 128] bf16.  Supported: page_size 16, 32, 64 or 128 tokens, D == 128; the three strides must be
 * multiples of 8 elements and k, v 16-byte aligned (tensor-map rules).  Slots that no logical
 * token maps to (tail of a last page, unreferenced pages) are never read into a result, but they
 * must hold finite bf16 values (they may pass through a multiply by an exactly zero weight).
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    const void* k;      /* device, bf16 */
    const void* v;      /* device, bf16 */
    int64_t num_pages;
    int32_t page_size;  /* 16, 32, 64 or 128 */
    int32_t Hkv;
    int32_t D;          /* 128 */
    int32_t reserved;
    int64_t stride_page, stride_tok, stride_head; /* elements */
} cp_kv_cache;

/* Workspace (device, 256-byte aligned) needed by the attention calls for a batch of B requests with
 * Hq query heads: the work lists of the persistent scheduler and the fp32 partial results of the
 * (query tile, head pair) units whose KV range is split over several CTAs for load balance (about
 * 55 MB of fixed partial space plus 16 bytes per unit).  new_len, C: host arrays of B entries.
 * Returns 0 on invalid arguments.  A workspace belongs to one call at a time: calls that may overlap on
 * the GPU (different streams without an ordering between them) need separate workspaces. */
size_t cp_workspace_bytes(int32_t B, const int64_t* new_len, const int32_t* C, int32_t Hq);

/* cp_schedule_inspect -- host only: the work distribution the attention calls would use for a batch
 * on a device with num_sms SMs (the varlen tile schedule: query tiles of 128 rows, the last tile of a
 * request possibly shorter -- a launch over all shards walks a request's rows as one run, so a tile may span
 * adjacent zigzag chunks but never two requests; one unit per tile and pair of query heads, or, when
 * Hq / Hkv is odd, per pair of consecutive tiles (256 rows) and single head; whole
 * units longest first -- KV head by KV head when the batch's K/V exceeds 32 MB, so that a long context's K/V
 * stays in L2 -- dealt to the CTAs in serpentine order, the remainder cut along KV so that every
 * CTA gets the same number of KV tile steps; when there are no more units than CTAs and all are short, every
 * unit gets a CTA of its own and nothing is cut).  summary (10 values): CTAs, query tiles, pieces, split units,
 * partial slots, largest / smallest per-CTA load in KV tile steps, their total, 1 if the work lists are small
 * enough to ride in the launch parameters, kernel launches the attention call makes (list copy unless they
 * ride along + attention + merge of split units if any).  pieces (optional,
 * 6 int32 per piece: cta, tile, head pair, first KV tile, end KV tile, partial slot or -1) and
 * items (optional, 4 int32 per tile: first packed row, rows, keys visible to the first row, KV tiles)
 * are filled when non-NULL and large enough (CP_ERR_WORKSPACE otherwise). */
int cp_schedule_inspect(int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                        int32_t Hq, int32_t Hkv, int32_t num_sms, int64_t* summary, int32_t* pieces,
                        int64_t max_pieces, int32_t* items, int64_t max_items);

/* ---------------------------------------------------------------------------------------------
 * cp_prefill_attn -- all C shards of one request in one launch (Sections 2.1-2.2).
 *   q          device [R, Hq, D] bf16, new tokens in original order
 *   page_table device int32, ceil((P+R)/page_size) entries, each in [0, num_pages) (the table lives
 *              on the device and is not validated; an entry outside the pool reads as zeros, it
 *              cannot fault)
 *   scale      softmax scale (1/sqrt(D) in the paper's definition)
 *   out        device [R, Hq, D] bf16; row r = softmax(scale * q_r K^T + mask) V, written at its
 *              original position (the "restore order" step is fused into the store)
 *   lse        device [Hq, R] fp32: natural-log sum-exp of the scaled scores of each row
 * The C shards of cp_plan(R, P, C) are row-disjoint and together cover all R rows (Section 2.1), and
 * adjacent chunks are adjacent rows with consecutive causal limits, so the launch walks the rows as one
 * run of 128-row query tiles with a per-row limit; C is validated, and the result does not depend on it
 * (the calls that compute ONE shard or ONE chunk cut their tiles at the chunk's boundaries).  Requires
 * Hq % Hkv == 0 (query head h uses KV head h / (Hq / Hkv)).  With an even group size a work unit is one
 * 128-row query tile for two query heads of a group, which share every K/V tile in shared memory; with an
 * odd one (e.g. Hq == Hkv) a unit is one head and two consecutive query tiles, which share the K/V tiles
 * the same way (measured on config 2's lengths: 1137 TFLOP/s with 16/16 heads against 1211 with 32/8).
 * One persistent launch computes all tiles; the few units that were split along KV to balance the SMs are
 * combined by a second small launch (an LSE merge of their partials).  Work lists of up to 24 KB travel in
 * the launch parameters; larger ones are first copied into the workspace by a small kernel.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 * ------------------------------------------------------------------------------------------- */
int cp_prefill_attn(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                    int64_t prefix_len, int64_t new_len, int32_t C, int32_t Hq, float scale,
                    void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream);

/* cp_prefill_attn_batch -- B requests in ONE launch (persistent varlen tile scheduler, longest
 * tiles first).  Host arrays: cu_new [B+1] (prefix sums of new_len; q/out rows of request b are
 * [cu_new[b], cu_new[b+1])), prefix_len [B], C [B], cu_pages [B+1] (request b's page table is
 * page_table[cu_pages[b] .. cu_pages[b+1]), with at least ceil((P_b+R_b)/page_size) entries).
 * q/out: device [cu_new[B], Hq, D] bf16; lse: device [Hq, cu_new[B]] fp32. */
int cp_prefill_attn_batch(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                          int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                          const int64_t* cu_pages, int32_t Hq, float scale, void* out, float* lse,
                          void* workspace, size_t workspace_bytes, void* stream);

/* cp_prefill_attn_shard -- only the rows of shard `shard` (0 <= shard < C) of cp_plan(R, P, C):
 * what one CP rank computes.  partial_out: device [R, Hq, D] fp32, partial_lse: device [Hq, R]
 * fp32; rows the shard does not own are written 0 with lse = -inf (by a spare warp of the same
 * launch), so that cp_merge over the C shard partials reproduces cp_prefill_attn exactly. */
int cp_prefill_attn_shard(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                          int64_t prefix_len, int64_t new_len, int32_t C, int32_t shard, int32_t Hq,
                          float scale, float* partial_out, float* partial_lse, void* workspace,
                          size_t workspace_bytes, void* stream);

/* cp_prefill_attn_chunk -- the rows of ONE zigzag chunk (0 <= chunk < 2C) of cp_plan(R, P, C), in
 * chunk-local buffers: what a CP rank runs twice per layer, once for its early chunk k as soon as the
 * keys of chunks 0..k have arrived and once for its late chunk 2C-1-k (Section 2.1: rank k holds the
 * k-th and (2C-1-k)-th chunks, gathers K/V, attends its local queries to all causally visible keys).
 *   q_chunk    device [n, Hq, D] bf16, n = rows of the chunk (q_end - q_begin of cp_plan); row i is
 *              new token q_begin + i, at absolute position P + q_begin + i
 *   out_chunk  device [n, Hq, D] bf16;  lse_chunk  device [Hq, n] fp32
 *   page_table device, ceil((P+R)/page_size) entries; only entries below ceil((P+q_end)/page_size)
 *              are read, later pages may still be empty.  Token slots of a referenced page that lie
 *              behind P + q_end are read and masked: they must hold finite values.
 * An empty chunk (padding of a short request) launches nothing and returns CP_OK.  Workspace as for
 * cp_prefill_attn with the same (R, C, Hq).  Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
int cp_prefill_attn_chunk(cp_ctx* ctx, const void* q_chunk, const cp_kv_cache* cache, const int32_t* page_table,
                          int64_t prefix_len, int64_t new_len, int32_t C, int32_t chunk, int32_t Hq,
                          float scale, void* out_chunk, float* lse_chunk, void* workspace,
                          size_t workspace_bytes, void* stream);

/* cp_prefill_attn_kvrange -- all R queries against the keys whose absolute position lies in
 * [kv_lo, kv_hi) only (still causal: new token r sees positions <= P + r): the partial result a CP rank
 * produces when the K/V stays sharded over the ranks and the queries travel instead (the alternative to
 * Section 2.1's all-gather when a worker's cached KV stays spread over its ranks, Section 2.2).  partial_out: device [R, Hq, D] fp32, normalised over the keys of the range; partial_lse:
 * device [Hq, R] fp32; a row that sees no key of the range gets zeros and lse = -inf.  Partials over
 * disjoint ranges that together cover [0, P + R) combine with cp_merge into cp_prefill_attn's result.
 * Only pages holding keys of the range are read.  kv_lo, kv_hi need no alignment.  Workspace as for
 * cp_prefill_attn with C = 1.  Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
int cp_prefill_attn_kvrange(cp_ctx* ctx, const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                            int64_t prefix_len, int64_t new_len, int64_t kv_lo, int64_t kv_hi, int32_t Hq,
                            float scale, float* partial_out, float* partial_lse, void* workspace,
                            size_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * cp_prefill_attn_static -- cp_prefill_attn for callers that must not allocate device memory.
 * (The paper has no counterpart to this call; it exists for integration reasons only.)
 * Who needs it: code that runs after an inference engine has handed all of HBM to its own KV-cache
 * pool, code inside a region where an allocation would synchronise the device or is forbidden
 * (a latency-critical serving loop, a library callback), and embedders that are simply not
 * allowed to create a cp_ctx, whose constructor allocates.  This call needs no cp_ctx and no
 * workspace, and it calls no allocating CUDA routine: the scheduler's tile list and the status
 * words live in a fixed device array of 65,792 bytes that is part of the library image (every GPU
 * that loads the library holds it until the process exits).
 *   - Same arguments, result and limits as cp_prefill_attn, computed on the CURRENT device.
 *   - Size limit: ceil(new_len / 128) must not exceed 2048 query tiles (262,144 new tokens);
 *     larger requests return CP_ERR_WORKSPACE and launch nothing.
 *   - Two launches on the given stream: a small kernel that clears the status words and writes
 *     the tile list from (new_len, prefix_len) passed by value, then the attention kernel.  No
 *     host buffer is read after the call returns.
 *   - The first call on each device resolves the device address of the array, the tensor-map
 *     encoder and the kernel's shared-memory attribute; make that first call before any stream
 *     capture begins.
 *   - All calls share the one array, which keeps the previous call's contents; the call clears
 *     the status words and rewrites the tile list in stream order.  Two calls that can overlap on
 *     the GPU (different streams without an ordering between them) race on it; host threads must
 *     not call it concurrently for the same device either.
 *   - A device-side wait that runs out is recorded in the array's status words, which this ABI
 *     does not expose; the rows of the affected tiles are then left unwritten.
 * ------------------------------------------------------------------------------------------- */
int cp_prefill_attn_static(const void* q, const cp_kv_cache* cache, const int32_t* page_table,
                           int64_t prefix_len, int64_t new_len, int32_t C, int32_t Hq, float scale,
                           void* out, float* lse, void* stream);

/* ---------------------------------------------------------------------------------------------
 * cp_merge -- N-way log-sum-exp combination of partial attention results over the same rows
 * (what joins per-shard or KV-split partials into full-sequence attention).  The paper states no
 * such step: its CP outputs are row-disjoint and are concatenated (Section 2.1).  This is the general
 * combine the library adds; row-disjoint shard partials (lse = -inf on rows a shard does not own) are
 * the special case that reproduces the paper's concatenation.
 *   partials device [N, T, H, D] fp32;  lses device [N, H, T] fp32 (natural log; -inf = "this
 *   partial holds nothing for the row": its values are ignored even if non-finite)
 *   out      device [T, H, D], bf16 or fp32 (out_dtype = CP_DTYPE_*)
 *   lse_out  device [H, T] fp32 or NULL
 * Per row: m = max_n lse_n; m = -inf -> out = 0, lse = -inf; else w_n = exp(lse_n - m),
 * out = sum w_n O_n / sum w_n, lse = m + ln sum w_n.  Supported: D == 128, 1 <= N <= 32.
 * ------------------------------------------------------------------------------------------- */
int cp_merge(cp_ctx* ctx, const float* partials, const float* lses, int32_t N, int64_t T, int32_t H,
             int32_t D, void* out, int32_t out_dtype, float* lse_out, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Paged <-> contiguous copies of n logical tokens starting at t_begin (the prefix-KV gather path
 * as a standalone op: Section 2.2 has the cached prefix KV resident at the worker, block by block;
 * the paper names no copy routine).  k_rows / v_rows: device [n, Hkv, D] bf16, contiguous.
 * page_table: device, at least ceil((t_begin + n) / page_size) entries, each in [0, num_pages).
 * Bit-exact copies.  Either of the k/v pairs may be NULL to copy only the other.  An entry outside
 * [0, num_pages) is never used as an address: the elements behind it are skipped (not read, not
 * written) and the first such entry is reported as CP_ERR_BOUNDS by cp_ctx_poll_status().
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA.
 * ------------------------------------------------------------------------------------------- */
int cp_kv_gather(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int64_t t_begin,
                 int64_t n, void* k_rows, void* v_rows, void* stream);
int cp_kv_append(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int64_t t_begin,
                 int64_t n, const void* k_rows, const void* v_rows, void* stream);

/* cp_check_page_table -- debug aid (the paper has no counterpart): enqueues a small kernel that compares every one of
 * the n_entries of a device page table with the pool size.  The table is only read.  After the stream has been
 * synchronised, cp_ctx_poll_status returns CP_ERR_BOUNDS with detail {code, index of the first bad entry found, block,
 * its page id} if an entry lies outside [0, num_pages).  The attention calls never fault on such an entry (the page
 * reads as zeros) and the copies skip it; this call is for finding it.  Errors: INVALID_ARG, CUDA. */
int cp_check_page_table(cp_ctx* ctx, const int32_t* page_table, int64_t n_entries, int64_t num_pages, void* stream);

/* cp_kv_append_segments -- cp_kv_append for several runs of rows in ONE launch: segment i writes rows
 * [row0, row0 + n) of k_rows / v_rows (device [*, Hkv, D] bf16) to logical tokens [t_begin, t_begin + n).  What a
 * CP rank needs after an all-gather of K and V (Section 2.1): the gathered blocks of the C ranks land at C
 * different token ranges of the rank's cache.  segments: host array; at most 64 segments per call; empty
 * segments are skipped.  Segments must not overlap in the cache.  Page ids are checked as in cp_kv_append.
 * Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
typedef struct {
    int64_t t_begin; /* first logical token written */
    int64_t n;       /* tokens */
    int64_t row0;    /* first row read from k_rows / v_rows */
} cp_kv_segment;
int cp_kv_append_segments(cp_ctx* ctx, const cp_kv_cache* cache, const int32_t* page_table, int32_t n_segments,
                          const cp_kv_segment* segments, const void* k_rows, const void* v_rows, void* stream);

/* ---------------------------------------------------------------------------------------------
 * FP8 K/V variant.  The paper's main model is an FP8 model (Section 9.1) but the paper states no FP8
 * attention recipe; the format below is this library's reading.
 *   - K and V pages hold OCP E4M3 bytes (1-4-3 bits, bias 7, no infinities, largest finite value 448),
 *     layout as cp_kv_cache with one byte per element (strides in bytes, multiples of 16); k_scale and
 *     v_scale are device arrays of Hkv fp32 values: the stored byte b of KV head g stands for
 *     scale[g] * e4m3(b).  Slots no logical token maps to must hold finite codes (not 0x7F / 0xFF).
 *   - Queries are bf16.  Each (token, head) row is quantised by a small pre-pass kernel: amax = max |q|,
 *     q_scale = amax / 448, code = e4m3(q * (448 / amax)), IEEE fp32 arithmetic, round to nearest even,
 *     saturating; a row of zeros has scale 0.
 *   - The result is the Section 2.1 formula (Section 2.2 prefix rule) on the dequantised values: Q K^T and
 *     P V run on the tensor cores with one-byte operands and fp32 accumulation; the softmax weights are
 *     rounded to E4M3 (after a scaling by 16) for P V, the row sum and the LSE use the unrounded weights.
 *     LSE is as accurate as in the bf16 path; each output element is within 2^-4 * sum_j p_j |v_j| of the
 *     exact result on the stored bytes (the rounding of the weights), typically 2-3 % of the row's norm.
 *   - out: bf16 [R, Hq, D]; lse: fp32 [Hq, R].
 * cp_workspace_bytes_fp8: the workspace of cp_workspace_bytes plus room for the quantised queries.
 * cp_kv_append_fp8: writes n logical tokens starting at t_begin from bf16 rows [n, Hkv, D] into the FP8
 * cache, each element as e4m3(x / scale[g]) (IEEE fp32 division, round to nearest even, saturating); page
 * ids outside the pool are skipped and reported as by cp_kv_append.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA.
 * ------------------------------------------------------------------------------------------- */
typedef struct {
    const void* k;          /* device, E4M3 bytes */
    const void* v;
    const float* k_scale;   /* device, [Hkv] fp32 */
    const float* v_scale;
    int64_t num_pages;
    int32_t page_size;      /* 16, 32, 64 or 128 */
    int32_t Hkv;
    int32_t D;              /* 128 */
    int32_t reserved;
    int64_t stride_page, stride_tok, stride_head; /* bytes */
} cp_kv_cache_fp8;
size_t cp_workspace_bytes_fp8(int32_t B, const int64_t* new_len, const int32_t* C, int32_t Hq);
int cp_prefill_attn_fp8(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                        int64_t prefix_len, int64_t new_len, int32_t C, int32_t Hq, float scale,
                        void* out, float* lse, void* workspace, size_t workspace_bytes, void* stream);
int cp_prefill_attn_fp8_batch(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                              int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                              const int64_t* cu_pages, int32_t Hq, float scale, void* out, float* lse,
                              void* workspace, size_t workspace_bytes, void* stream);
/* The one-shard, one-chunk and key-range forms of the FP8 variant: arguments, tile lists, fill of uncovered rows and
 * results as in cp_prefill_attn_shard / _chunk / _kvrange, on an FP8 cache (partials in fp32, ready for cp_merge);
 * workspace as cp_workspace_bytes_fp8 says. */
int cp_prefill_attn_fp8_shard(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                              int64_t prefix_len, int64_t new_len, int32_t C, int32_t shard, int32_t Hq,
                              float scale, float* partial_out, float* partial_lse, void* workspace,
                              size_t workspace_bytes, void* stream);
int cp_prefill_attn_fp8_chunk(cp_ctx* ctx, const void* q_chunk, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                              int64_t prefix_len, int64_t new_len, int32_t C, int32_t chunk, int32_t Hq,
                              float scale, void* out_chunk, float* lse_chunk, void* workspace,
                              size_t workspace_bytes, void* stream);
int cp_prefill_attn_fp8_kvrange(cp_ctx* ctx, const void* q, const cp_kv_cache_fp8* cache, const int32_t* page_table,
                                int64_t prefix_len, int64_t new_len, int64_t kv_lo, int64_t kv_hi, int32_t Hq,
                                float scale, float* partial_out, float* partial_lse, void* workspace,
                                size_t workspace_bytes, void* stream);
int cp_kv_append_fp8(cp_ctx* ctx, const cp_kv_cache_fp8* cache, const int32_t* page_table, int64_t t_begin,
                     int64_t n, const void* k_rows, const void* v_rows, void* stream);
/* Raw byte copies of an FP8 cache, no conversion: cp_kv_gather_fp8 reads n logical tokens from t_begin into
 * k_bytes / v_bytes (device [n, Hkv, D] E4M3 bytes); cp_kv_append_segments_fp8 writes runs of such rows like
 * cp_kv_append_segments.  For the exchange between CP ranks whose caches share the per-head scales: the stored
 * bytes travel (half of what bf16 rows cost on the link) and are appended as they are.  Bit-exact; page ids are
 * checked as in cp_kv_append.  Errors: INVALID_ARG, UNSUPPORTED, CUDA. */
int cp_kv_gather_fp8(cp_ctx* ctx, const cp_kv_cache_fp8* cache, const int32_t* page_table, int64_t t_begin,
                     int64_t n, void* k_bytes, void* v_bytes, void* stream);
int cp_kv_append_segments_fp8(cp_ctx* ctx, const cp_kv_cache_fp8* cache, const int32_t* page_table, int32_t n_segments,
                              const cp_kv_segment* segments, const void* k_bytes, const void* v_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* CPATTN_H */

// Cache-aware causal prefill attention for sm_100a: tcgen05 tensor cores with TMEM accumulators,
// TMA-staged Q/K/V tiles (K/V fetched page by page through the page table), online softmax.
//
// One persistent CTA per SM walks a list of work units.  A unit is one query tile (<= 128 new
// tokens) for TWO query heads of the same KV group, so each K/V tile that lands in shared memory
// feeds two 128x128 score tiles (GQA head sharing).  With an odd group size (plain multi-head
// attention, for instance) a unit is ONE query head and TWO consecutive query tiles (<= 256 new tokens):
// the two tiles share every K/V tile the same way, the later one seeing one more KV tile at the end,
// which is fully masked for the earlier one ("tile-pair" units).  Warp roles:
//   warps 0-3  softmax warpgroup for head 0 of the pair (tile-pair units: rows 0-127): one thread per query row
//   warps 4-7  softmax warpgroup for head 1 (tile-pair units: rows 128-255)
//   warp  8    TMA producer (the warp prefetches page ids; the pages of a tile go out from several lanes)
//              (with 16-token pages the spare warp copies the second 64-dim half of every K/V tile)
//   warp  9    tcgen05.mma issuer for the scores S = Q K^T (warp-uniform loop, one elected lane issues)
//   warp  10   tcgen05.mma issuer for O += P V
//   warp  11   spare (completes the third warpgroup so that register budgets can be moved: the softmax
//              warpgroups run with 200 registers per thread, the third one with 104); in the calls that
//              produce partial results it writes zeros / -inf into the rows the call does not compute
// TMEM (512 columns): S | P0 | P1 | O0 | O1.  S is ONE score buffer (128 fp32 columns) that the two heads
// use in turn; P (bf16, 64 columns per head) is the TMEM A operand of P*V; O0, O1 are the accumulators.
// A softmax warpgroup reads its score tile into registers and hands the buffer back at once, so the next
// score tile -- the other head's, then its own next one -- is computed while it exponentiates: in steady
// state no softmax warpgroup waits for the tensor pipe, and both MUFU and tensor pipe stay about 74 % busy.
// The two issuers need no ordering between them (disjoint TMEM, separate barriers for K and V tiles).
// P is handed over in two pieces (96 keys, then 32), so P*V starts while the rest of the row is still
// being exponentiated.
// Every wait is bounded; on expiry the CTA records where it gave up in the status word, all roles
// drain and the kernel returns normally.
#pragma once

#include <cuda_bf16.h>

#include <algorithm>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "internal.h"

using namespace cpattn;

namespace {

constexpr int kD = 128;
constexpr int kBlockM = 128;
constexpr int kBlockN = 128;
constexpr int kKvStages = 5;                       // ring of 32 KB tiles, K and V alternate
constexpr uint32_t kTileBytes = kBlockN * kD * 2;  // 32768
constexpr uint32_t kHalfBytes = kTileBytes / 2;    // one 64-dim half: 128 rows x 128 B
constexpr int kThreads = 384;
// setmaxnreg budgets after the role split.  Their total must stay below the 64K register file by at
// least one allocation step: with a split that used the whole file (208 / 96) the softmax warps never got
// their registers and the kernel did not start its work.
constexpr int kRegsSoftmax = 200;
constexpr int kRegsOther = 104;
static_assert(2 * 128 * kRegsSoftmax + 128 * kRegsOther <= 65536 - 1024, "leave slack in the register file");

// shared memory map (offsets from a 1024-byte aligned base)
constexpr uint32_t kSmemQ = 0;                                  // 2 heads x 32 KB
constexpr uint32_t kSmemKV = 2 * kTileBytes;                    // kKvStages x 32 KB
constexpr uint32_t kSmemBar = kSmemKV + kKvStages * kTileBytes; // mbarriers
constexpr uint32_t kSmemBytes = kSmemBar + 256;
constexpr uint32_t kSmemAlloc = kSmemBytes + 1024;              // slack for manual alignment

// barrier indices (8 bytes each, from kSmemBar); also the ids reported on a timeout
enum Bar : uint32_t {
    kBarQFull = 0, kBarQEmpty = 1,
    kBarKvFull = 2,                       // + stage
    kBarKvEmpty = kBarKvFull + kKvStages, // + stage
    kBarSReady = kBarKvEmpty + kKvStages, // + wg: the score tile in the S buffer belongs to this head and is complete
    kBarSFree = kBarSReady + 2,           // the S buffer has been read into registers (one phase per score tile)
    kBarPReady = kBarSFree + 1,           // + wg*4 + piece
    kBarPvDone = kBarPReady + 8,          // + wg: P*V of a tile has finished (P and O of the head may be touched)
    kBarOFree = kBarPvDone + 2,           // + wg
    kNumBars = kBarOFree + 2
};
static_assert(kNumBars * 8 + 16 <= 256, "barrier area");
constexpr uint32_t kSmemTmemPtr = kSmemBar + kNumBars * 8;      // uint32: TMEM base address
constexpr uint32_t kSmemAbort = kSmemTmemPtr + 4;               // uint32: set when a wait expired

// TMEM columns
constexpr uint32_t kTmemS = 0;     // one score tile (fp32), shared by the two heads in turn
constexpr uint32_t kTmemP = 128;   // + wg * 64: P of a head (bf16), the TMEM A operand of P*V
constexpr uint32_t kTmemO = 256;   // + wg * 128

constexpr uint32_t kTryWaitHintNs = 200000;             // the thread may stay suspended this long per try
constexpr long long kWaitLimitCycles = 4000000000ll;   // about two seconds
constexpr float kRescaleThreshold = 8.0f;
// FP8 K/V variant: one K or V tile is 128 keys x 128 one-byte elements (it uses the first half of a 32 KB ring
// slot); P is multiplied by 2^kP8Shift before it is rounded to E4M3, and the running-max reference may lag by at
// most 2^kRescaleThreshold8, so that the scaled weights stay <= 256 (the format ends at 448) while weights down
// to 2^-10 of the row's largest keep the full 3-bit mantissa.
constexpr uint32_t kTileBytes8 = kBlockN * kD;     // 16384
constexpr float kRescaleThreshold8 = 4.0f;
constexpr float kP8Shift = 4.0f;
constexpr int kPieces = 2;                            // P is handed to the P*V issuer in two pieces:
constexpr int kSplitQ = 3;                            // the first kSplitQ quarters of the row, then the rest
constexpr int kPolyOf4 = 0;                            // pairs out of every four whose exp2 runs on the FMA pipe instead of MUFU:
                                                       // 0 since both softmax warpgroups run all the time (issue slots are the
                                                       // scarcer resource: 1 costs 3 %, 2 costs 12 %); 1 was best while they alternated

struct AttnParams {
    const TileItem* items;
    int32_t n_items;
    const int32_t* cta_off;    // explicit schedule: pieces of CTA b are pieces[cta_off[b] .. cta_off[b+1]);
    const PieceEntry* pieces;  // NULL: implicit serpentine schedule over whole units (no KV splits)
    float* partial_o;          // [slots][2 heads][128 rows][128] fp32, normalised partial outputs
    float* partial_lse;        // [slots][2 heads][128 rows]
    int32_t pairs_per_tile;   // units per query tile: Hq / heads_per_unit
    int32_t pairs_per_kv;     // implicit schedule: > 0 walks the units KV head by KV head (this many units per tile and KV head)
    int32_t heads_per_unit;   // 2: two query heads of one KV group share every K/V tile; 1: odd group size, the unit
                              // is one head and two consecutive 128-row query tiles (tile-pair unit)
    int32_t group;            // Hq / Hkv
    int32_t Hq;
    const int32_t* page_table;
    int32_t oob_page;         // a page coordinate outside the tensor map: TMA fills zeros
    int32_t page_tokens;      // tokens per page: 16, 32, 64 or 128 (one TMA box = one page x 64 dims)
    float scale_log2;         // scale * log2(e)
    void* out;
    int32_t out_f32;          // 0: bf16 [rows, Hq, D]; 1: fp32
    float* lse;
    int64_t lse_stride;       // total rows
    int32_t* status;
    // byte offsets of items / cta_off / pieces inside the launch-parameter copy of a small schedule; < 0: the
    // lists are in global memory behind the pointers above
    int32_t inl_items, inl_cta_off, inl_pieces;
    // partial-result calls: row ranges [fill[2i], fill[2i+1]) that no tile covers get zeros (out, fp32) and
    // lse = -inf from the kernel's spare warp
    int32_t n_fill;
    int32_t fill[2 * kMaxFillRanges];
    // FP8 K/V variant: per-row query scales [rows, Hq] (written by the quantising pre-pass), per-KV-head scales
    const float* q_scale;
    const float* k_scale;
    const float* v_scale;
    int32_t co_producer;      // 1: the spare warp copies the second 64-dim half of every K/V tile (16-token pages, bf16)
};

// ------------------------------------------------------------------------------------------
// PTX wrappers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity), "r"(kTryWaitHintNs) : "memory");
    return ok != 0;
}

// Non-blocking test of a phase; the result comes back asynchronously, so a test issued before a block
// of MMAs costs nothing by the time it is looked at.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2,
                                            int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

// True in exactly one lane of the (converged) warp.
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "elect.sync _|p, 0xffffffff;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

// the same two forms for one-byte operands (E4M3 x E4M3, fp32 accumulation; K = 32 per instruction)
__device__ __forceinline__ void mma_ss_f8(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}
__device__ __forceinline__ void mma_ts_f8(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(acc) : "memory");
}

#define CP_R8(a, o) "=f"(a[o + 0]), "=f"(a[o + 1]), "=f"(a[o + 2]), "=f"(a[o + 3]), "=f"(a[o + 4]), "=f"(a[o + 5]), "=f"(a[o + 6]), "=f"(a[o + 7])
#define CP_W8F(a, o) "f"(a[o + 0]), "f"(a[o + 1]), "f"(a[o + 2]), "f"(a[o + 3]), "f"(a[o + 4]), "f"(a[o + 5]), "f"(a[o + 6]), "f"(a[o + 7])
#define CP_W8R(a, o) "r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]), "r"(a[o + 7])

// 32 consecutive fp32 columns of this thread's TMEM lane -> registers v[o .. o+31]
#define TMEM_LD32(taddr, v, o)                                                                            \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "                                                \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                  \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"                 \
                 : CP_R8(v, o), CP_R8(v, o + 8), CP_R8(v, o + 16), CP_R8(v, o + 24) : "r"(taddr) : "memory")
#define TMEM_ST32F(taddr, v, o)                                                                           \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                         \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                  \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"                        \
                 ::CP_W8F(v, o), CP_W8F(v, o + 8), CP_W8F(v, o + 16), CP_W8F(v, o + 24), "r"(taddr) : "memory")
#define TMEM_ST16R(taddr, v, o)                                                                           \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%16], "                                         \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15};"                                 \
                 ::CP_W8R(v, o), CP_W8R(v, o + 8), "r"(taddr) : "memory")
#define TMEM_ST8R(taddr, v, o)                                                                            \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%8], {%0,%1,%2,%3,%4,%5,%6,%7};"                    \
                 ::CP_W8R(v, o), "r"(taddr) : "memory")
#define TMEM_ST32R(taddr, v, o)                                                                           \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%32], "                                         \
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"                                  \
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31};"                        \
                 ::CP_W8R(v, o), CP_W8R(v, o + 8), CP_W8R(v, o + 16), CP_W8R(v, o + 24), "r"(taddr) : "memory")

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float lg2(float x) {
    float y;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
// 2^x for a pair of arguments x <= 0 on the FMA pipe (no MUFU): round to nearest integer with the
// 1.5*2^23 trick, cubic minimax polynomial of 2^f on [-0.5, 0.5] (relative error 7.5e-5, far below
// the bf16 rounding of P), integer part added into the exponent field.
__device__ __forceinline__ float2 ex2_poly2(float2 x) {
    const float kMagic = 12582912.f;
    x.x = fmaxf(x.x, -126.f);
    x.y = fmaxf(x.y, -126.f);
    const float2 r = __fadd2_rn(x, make_float2(kMagic, kMagic));
    const float2 xi = __fadd2_rn(r, make_float2(-kMagic, -kMagic));
    const float2 f = __fadd2_rn(x, make_float2(-xi.x, -xi.y));
    float2 p = __ffma2_rn(f, make_float2(0.0551716648f, 0.0551716648f), make_float2(0.2426111251f, 0.2426111251f));
    p = __ffma2_rn(p, f, make_float2(0.6932609677f, 0.6932609677f));
    p = __ffma2_rn(p, f, make_float2(0.9999280572f, 0.9999280572f));
    float2 out;
    out.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(r.x) << 23));
    out.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(r.y) << 23));
    return out;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&b);
}

// Four weights -> four E4M3 bytes of one TMEM column, lowest key in the lowest byte (round to nearest even,
// saturating at 448).  cvt packs its first source into the upper byte of the pair.
__device__ __forceinline__ uint32_t pack_e4m3x4(float e0, float e1, float e2, float e3) {
    uint16_t lo, hi;
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(lo) : "f"(e1), "f"(e0));
    asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(hi) : "f"(e3), "f"(e2));
    return (uint32_t)lo | ((uint32_t)hi << 16);
}

// tcgen05 shared-memory matrix descriptor, 128-byte swizzle (layout type 2), descriptor version 1.
// K-major operand (Q, K): rows of 128 B, 8-row groups 1024 B apart (SBO); LBO unused.
// MN-major operand (V): 64 dims contiguous per key row (128 B), 8-key groups 1024 B apart (SBO),
// the next 64 dims one half-tile (16 KB) further (LBO).
__device__ __forceinline__ uint64_t make_desc(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)(lbo_bytes >> 4) << 16;
    d |= (uint64_t)(sbo_bytes >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}

// instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = 128; bit 16 = B is MN-major
constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((kBlockN >> 3) << 17) | ((kBlockM >> 4) << 24);
constexpr uint32_t kIdescPV = kIdescS | (1u << 16);
// one-byte operands: A and B format fields 0 = E4M3; same shape; K = 32 per instruction
constexpr uint32_t kIdescS8 = (1u << 4) | ((kBlockN >> 3) << 17) | ((kBlockM >> 4) << 24);
constexpr uint32_t kIdescPV8 = kIdescS8 | (1u << 16);

// Bounded wait on an mbarrier phase.  The fast path is a single try; the slow path spins with a cycle
// limit.  When the limit runs out the first thread to notice records {code, barrier id, block,
// iteration} in the status word and raises the CTA's abort flag; from then on every wait of the CTA
// gives up after one failed try, so all roles run off the end of their loops without blocking (the
// results are garbage, the status word says so) and the kernel returns normally.
__device__ __forceinline__ void mbar_wait(uint32_t bar_base, uint32_t bar_id, uint32_t parity, volatile uint32_t* abort_flag,
                                          int32_t* status, int iter, long long limit_cycles = kWaitLimitCycles) {
    const uint32_t bar = bar_base + bar_id * 8;
    if (mbar_try_wait(bar, parity)) return;
    const long long t0 = clock64();
    while (true) {
        if (*abort_flag) return;
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return;
        if (clock64() - t0 > limit_cycles) {
            *abort_flag = 1;
            if (atomicCAS(status, 0, CP_ERR_TIMEOUT) == 0) {
                status[1] = (int32_t)bar_id;
                status[2] = (int32_t)blockIdx.x;
                status[3] = iter;
            }
            return;
        }
    }
}

// One piece of work of a CTA: KV tiles [t_begin, t_end) of one query tile for one pair of heads.
struct UnitInfo {
    TileItem it;
    int head0;
    int kv_head;
    int t_begin, t_end;   // KV tile range of this piece
    int slot;             // < 0: whole unit, final rows; >= 0: partial slot
};

// Two schedules.  Explicit (p.pieces != NULL): the host lists, per CTA, whole units and the KV
// ranges of units that were split to fill every CTA to the same number of KV tile steps.  Implicit:
// serpentine over the longest-first unit list -- in even rounds CTA c takes unit round*grid + c, in
// odd rounds round*grid + (grid-1-c), which evens out the sorted lengths; whole units only.
__device__ __forceinline__ bool fetch_unit(const AttnParams& p, const InlineSched& inl, int round, UnitInfo& u) {
    int item, pair;
    // a small schedule sits in the launch parameters (constant bank), a large one in the workspace
    const TileItem* items = p.inl_items >= 0 ? reinterpret_cast<const TileItem*>(inl.bytes + p.inl_items) : p.items;
    if (p.pieces != nullptr || p.inl_pieces >= 0) {
        const int32_t* cta_off = p.inl_cta_off >= 0 ? reinterpret_cast<const int32_t*>(inl.bytes + p.inl_cta_off) : p.cta_off;
        const PieceEntry* pieces = p.inl_pieces >= 0 ? reinterpret_cast<const PieceEntry*>(inl.bytes + p.inl_pieces) : p.pieces;
        const int idx = cta_off[blockIdx.x] + round;
        if (idx >= cta_off[blockIdx.x + 1]) return false;
        const PieceEntry e = pieces[idx];
        item = e.item;
        pair = e.pair;
        u.t_begin = e.t_begin;
        u.t_end = e.t_end;
        u.slot = e.slot;
        u.it = items[item];
    } else {
        const int g = gridDim.x;
        const int c = (round & 1) ? (g - 1 - (int)blockIdx.x) : (int)blockIdx.x;
        const int64_t idx = (int64_t)round * g + c;
        const int64_t total = (int64_t)p.n_items * p.pairs_per_tile;
        if (idx >= total) return false;
        if (p.pairs_per_kv > 0) {
            // KV head by KV head: all CTAs read one head's K/V at a time (a long context then stays in L2)
            const int64_t per_head = (int64_t)p.n_items * p.pairs_per_kv;
            const int g = (int)(idx / per_head);
            const int64_t rem = idx - (int64_t)g * per_head;
            item = (int)(rem / p.pairs_per_kv);
            pair = g * p.pairs_per_kv + (int)(rem - (int64_t)item * p.pairs_per_kv);
        } else {
            item = (int)(idx / p.pairs_per_tile);
            pair = (int)(idx - (int64_t)item * p.pairs_per_tile);
        }
        u.it = items[item];
        u.t_begin = 0;
        u.t_end = u.it.n_kv_tiles;
        u.slot = -1;
    }
    const int t0 = u.it.kv_lo >> 7;      // first KV tile of the unit's key range (0 for the ordinary calls)
    u.t_begin += t0;
    u.t_end += t0;
    u.head0 = p.heads_per_unit * pair;
    u.kv_head = u.head0 / p.group;
    return true;
}

// ------------------------------------------------------------------------------------------
// Roles
// ------------------------------------------------------------------------------------------
// half_lo, half_hi: the 64-dim halves of every K/V tile this warp copies.  Normally warp 8 copies both; with
// 16-token pages (sixteen 2 KB boxes per tile, whose issue cost a single warp cannot hide) the spare warp takes
// the second half as a co-producer: it waits for the same "slot empty" phases, while the byte count of a tile is
// announced once, by the leading warp (a copy that lands before the announcement only leaves the barrier's byte
// count negative for a moment; the phase cannot complete before the announcing arrival).
template <bool kFp8>
__device__ __forceinline__ void producer_role(const CUtensorMap* tmQ, const CUtensorMap* tmK, const CUtensorMap* tmV, const AttnParams& p,
                              const InlineSched& inl, uint32_t smem_base, volatile uint32_t* abort_flag, int half_lo,
                              int half_hi) {
    const int lane = threadIdx.x & 31;
    const uint32_t bars = smem_base + kSmemBar;
    const bool lead = half_lo == 0;
    uint32_t kv_it = 0;   // ring slots filled so far
    for (int round = 0;; ++round) {
        UnitInfo u;
        if (!fetch_unit(p, inl, round, u)) break;
        if (lane == 0 && lead) {
            mbar_wait(bars, kBarQEmpty, (round & 1) ^ 1, abort_flag, p.status, round);
            const uint32_t qbar = bars + kBarQFull * 8;
            mbar_expect_tx(qbar, 2 * (kFp8 ? kTileBytes8 : kTileBytes));
            for (int h = 0; h < 2; ++h) {
                // second Q tile: the next head of the pair, or (tile-pair unit) the next 128 rows of the same head
                const int head = u.head0 + (p.heads_per_unit == 2 ? h : 0);
                const int row0 = u.it.q_row0 + (p.heads_per_unit == 2 ? 0 : h * kBlockM);
                if (kFp8) {      // one-byte queries: a row is one 128-byte swizzle line
                    tma_load_3d(smem_base + kSmemQ + h * kTileBytes, tmQ, qbar, 0, head, row0);
                } else {
                    for (int half = 0; half < 2; ++half)
                        tma_load_3d(smem_base + kSmemQ + h * kTileBytes + half * kHalfBytes, tmQ, qbar, half * 64, head, row0);
                }
            }
        }
        __syncwarp();
        const int n_tiles = u.t_end;
        const int ppt = kBlockN / p.page_tokens;          // pages per KV tile: 8, 4, 2 or 1
        const uint32_t box_bytes = (uint32_t)p.page_tokens * 128u;   // one page x 64 bf16 dims (x 128 one-byte dims)
        // load order = order of first use by the issuers: K(j0), then K(j+1) before V(j)
        const int n_loads = 2 * (n_tiles - u.t_begin);
        int pg_base = -1;       // first page whose id the lanes currently hold
        int my_page = 0;
        for (int ld = 0; ld < n_loads; ++ld) {
            // ld 0: K(j0); odd ld: K(j0 + (ld+1)/2) except the last, which is V(n-1); even ld > 0: V(j0 + ld/2 - 1)
            int j, kv;
            if (ld == 0) { j = u.t_begin; kv = 0; }
            else if (ld == n_loads - 1) { j = n_tiles - 1; kv = 1; }
            else if (ld & 1) { j = u.t_begin + (ld + 1) / 2; kv = 0; }
            else { j = u.t_begin + ld / 2 - 1; kv = 1; }
            const int pg0 = ppt * j;
            if (pg_base < 0 || pg0 < pg_base || pg0 + ppt > pg_base + 32) {
                // the warp fetches 32 page ids starting at this tile (K runs one tile ahead of V, so the
                // window is anchored at the V tile when possible)
                pg_base = ppt * max(j - 1, u.t_begin);
                const int pg = pg_base + lane;
                my_page = (pg < u.it.n_pages) ? __ldg(p.page_table + u.it.pt_base + pg) : p.oob_page;
            }
            const uint32_t slot = kv_it % kKvStages;
            const uint32_t fbar = bars + (kBarKvFull + slot) * 8;
            const uint32_t dst = smem_base + kSmemKV + slot * kTileBytes;
            const CUtensorMap* map = kv ? tmV : tmK;
            if (lane == 0) {
                mbar_wait(bars, kBarKvEmpty + slot, ((kv_it / kKvStages) & 1) ^ 1, abort_flag, p.status, j);
                if (lead) mbar_expect_tx(fbar, kFp8 ? kTileBytes8 : kTileBytes);
            }
            __syncwarp();
            // lane i < ppt copies page i of the tile: this warp's 64-dim halves of its box (one-byte tiles have one)
            const int page = __shfl_sync(0xffffffffu, my_page, (pg0 - pg_base + (lane < ppt ? lane : 0)) & 31);
            if (lane < ppt) {
                for (int half = half_lo; half < (kFp8 ? 1 : half_hi); ++half)
                    tma_load_4d(dst + half * kHalfBytes + lane * box_bytes, map, fbar, half * 64, u.kv_head, 0, page);
            }
            __syncwarp();
            ++kv_it;
        }
    }
}

// The issuer warp.  One score buffer S serves both heads in turn, P and O have their own TMEM columns per
// head.  A score tile is read into registers by its softmax warpgroup as soon as that group is free, and
// the next score tile (of the other head, or of the same head when a unit has one) is issued the moment
// the buffer has been read -- so the scores of a head's next tile are computed while the head is still
// exponentiating the current one, and a softmax warpgroup never waits for the tensor pipe in steady state.
// With H heads per unit and tiles numbered S_0, S_1, ... (head fastest), P_k = P*V of tile k, the issue
// order is S_0 .. S_H, then P_k followed by S_(k+H+1).  P arrives in two pieces (96 keys, then 32).
// The whole warp runs the loop (waits included) so that addresses stay warp-uniform; one elected lane issues.
// Position in the K/V ring: slot and phase parity, advanced without divisions.
struct RingPos {
    uint32_t slot, par;
    __device__ __forceinline__ RingPos plus(uint32_t n) const {   // n < kKvStages
        RingPos r = {slot + n, par};
        if (r.slot >= (uint32_t)kKvStages) { r.slot -= kKvStages; r.par ^= 1u; }
        return r;
    }
};

// Two issuer warps, one per kind of product; nothing orders them against each other, because score tiles
// (S buffer) and P*V (P and O columns) touch disjoint TMEM and the K and V tiles have their own barriers.
//
// Score issuer: S tiles in the order (tile, head); each needs its K tile and the buffer back (s_free).
template <bool kFp8>
__device__ __forceinline__ void mma_s_role(const AttnParams& p, const InlineSched& inl, uint32_t smem_base, uint32_t tmem_base,
                                           volatile uint32_t* abort_flag) {
    const uint32_t bars = smem_base + kSmemBar;
    constexpr int H = 2;
    RingPos unit_pos = {0, 0};         // ring position of the unit's first load, K(j0)
    uint32_t s_par = 1;                // parity of "previous score tile was read"; 1: no tile yet (passes)
    const uint64_t q_desc0 = make_desc(smem_base + kSmemQ, 16, 1024);
    const uint64_t k_desc0 = make_desc(smem_base + kSmemKV, 16, 1024);           // K-major view of a ring slot
    // the next unit's description is fetched while the current one runs (three dependent loads otherwise sit between
    // the last score tile of a unit and the first of the next)
    UnitInfo u, nu;
    bool have = fetch_unit(p, inl, 0, u);
    for (int round = 0; have; ++round) {
        const bool have_next = fetch_unit(p, inl, round + 1, nu);
        const int j0 = u.t_begin, n = u.t_end;
        mbar_wait(bars, kBarQFull, round & 1, abort_flag, p.status, round);
        RingPos kpos = unit_pos;
#pragma unroll 1
        for (int j = j0; j < n; ++j) {
            mbar_wait(bars, kBarKvFull + kpos.slot, kpos.par, abort_flag, p.status, j);
            for (int h = 0; h < H; ++h) {
                const int wgt = h;
                mbar_wait(bars, kBarSFree, s_par, abort_flag, p.status, j);
                s_par ^= 1u;
                tc_fence_after();
                if (elect_one()) {
                    if (kFp8) {
                        // one-byte operands: the 128 dims of a row are one swizzle line, four steps of 32 bytes
#pragma unroll
                        for (int ks = 0; ks < kD / 32; ++ks)
                            mma_ss_f8(tmem_base + kTmemS, q_desc0 + (h * (kTileBytes >> 4)) + ks * 2,
                                      k_desc0 + kpos.slot * (kTileBytes >> 4) + ks * 2, kIdescS8, ks > 0);
                    } else {
#pragma unroll
                        for (int ks = 0; ks < kD / 16; ++ks) {
                            const uint32_t off = ((ks >> 2) * kHalfBytes + (ks & 3) * 32) >> 4;
                            mma_ss(tmem_base + kTmemS, q_desc0 + (h * (kTileBytes >> 4)) + off,
                                   k_desc0 + kpos.slot * (kTileBytes >> 4) + off, kIdescS, ks > 0);
                        }
                    }
                    tc_commit(bars + (kBarSReady + wgt) * 8);
                    if (h == H - 1) {
                        tc_commit(bars + (kBarKvEmpty + kpos.slot) * 8);
                        if (j == n - 1) tc_commit(bars + kBarQEmpty * 8);
                    }
                }
                __syncwarp();
            }
            kpos = kpos.plus(j == j0 ? 1 : 2);     // load order: K(j0), K(j0+1), V(j0), K(j0+2), V(j0+1), ...
        }
        const uint32_t adv = (uint32_t)(2 * (n - j0));
        const uint32_t q5 = adv / kKvStages, r5 = adv - q5 * kKvStages;
        unit_pos = unit_pos.plus(r5);
        unit_pos.par ^= (q5 & 1u);
        u = nu;
        have = have_next;
    }
}

// P*V issuer: O_h += P_h V_j in the order (tile, head), each in the two pieces P is handed over in.  In a
// single-head unit (a pair of consecutive query tiles of one head) the second P / O column set belongs to the
// unit's second query tile instead of a second head; the loop is the same.
template <bool kFp8>
__device__ __forceinline__ void mma_pv_role(const AttnParams& p, const InlineSched& inl, uint32_t smem_base, uint32_t tmem_base,
                                            volatile uint32_t* abort_flag) {
    const uint32_t bars = smem_base + kSmemBar;
    constexpr int H = 2;
    RingPos unit_pos = {0, 0};
    uint32_t p_par0 = 0, p_par1 = 0;   // phase parity of p_ready per softmax warpgroup
    const uint64_t v_desc0 = make_desc(smem_base + kSmemKV, kHalfBytes, 1024);   // MN-major view of a ring slot
    UnitInfo u, nu;
    bool have = fetch_unit(p, inl, 0, u);
    for (int round = 0; have; ++round) {
        const bool have_next = fetch_unit(p, inl, round + 1, nu);      // fetched ahead, as in the score issuer
        const int j0 = u.t_begin, n = u.t_end;
        RingPos vpos = unit_pos.plus(n - j0 == 1 ? 1 : 2);   // V(j0)
#pragma unroll 1
        for (int j = j0; j < n; ++j) {
            mbar_wait(bars, kBarKvFull + vpos.slot, vpos.par, abort_flag, p.status, j);
            for (int h = 0; h < H; ++h) {
                const int wgt = h;                 // P / O column set and softmax warpgroup
                const bool first = j == j0;        // first tile of this accumulator in the unit
                if (first && round > 0) mbar_wait(bars, kBarOFree + wgt, (round - 1) & 1, abort_flag, p.status, j);
                const uint32_t ppar = wgt ? p_par1 : p_par0;
#pragma unroll
                for (int part = 0; part < kPieces; ++part) {
                    mbar_wait(bars, kBarPReady + wgt * 4 + part, ppar, abort_flag, p.status, j);
                    tc_fence_after();
                    if (elect_one()) {
                        if (kFp8) {
                            // P in E4M3: 4 keys per TMEM column, 32 keys (8 columns, 32 V rows of 128 B) per instruction
                            const int ks0 = part == 0 ? 0 : kSplitQ, ks1 = part == 0 ? kSplitQ : 4;
#pragma unroll
                            for (int ks = 0; ks < 4; ++ks) {
                                if (ks >= ks0 && ks < ks1)
                                    mma_ts_f8(tmem_base + kTmemO + wgt * 128, tmem_base + kTmemP + wgt * 64 + ks * 8,
                                              v_desc0 + vpos.slot * (kTileBytes >> 4) + ks * (4096 >> 4), kIdescPV8,
                                              !first || ks > 0);
                            }
                        } else {
                        const int ks0 = part == 0 ? 0 : 2 * kSplitQ, ks1 = part == 0 ? 2 * kSplitQ : 8;
#pragma unroll
                        for (int ks = 0; ks < 8; ++ks) {
                            if (ks >= ks0 && ks < ks1)
                                mma_ts(tmem_base + kTmemO + wgt * 128, tmem_base + kTmemP + wgt * 64 + ks * 8,
                                       v_desc0 + vpos.slot * (kTileBytes >> 4) + ks * (2048 >> 4), kIdescPV,
                                       !first || ks > 0);
                        }
                        }
                        if (part == kPieces - 1) {
                            tc_commit(bars + (kBarPvDone + wgt) * 8);
                            if (h == H - 1) tc_commit(bars + (kBarKvEmpty + vpos.slot) * 8);
                        }
                    }
                    __syncwarp();
                }
                if (wgt) p_par1 ^= 1u; else p_par0 ^= 1u;
            }
            vpos = vpos.plus(j + 2 == n ? 1 : 2);
        }
        const uint32_t adv = (uint32_t)(2 * (n - j0));
        const uint32_t q5 = adv / kKvStages, r5 = adv - q5 * kKvStages;
        unit_pos = unit_pos.plus(r5);
        unit_pos.par ^= (q5 & 1u);
        u = nu;
        have = have_next;
    }
}

// Row max of 32 raw scores into four independent chains.
__device__ __forceinline__ void max32(const float (&s)[32], float& a0, float& a1, float& a2, float& a3) {
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
        a0 = max3(a0, s[i], s[i + 1]);
        a1 = max3(a1, s[i + 2], s[i + 3]);
        a2 = max3(a2, s[i + 4], s[i + 5]);
        a3 = max3(a3, s[i + 6], s[i + 7]);
    }
}
// Columns at or beyond `lim` are above the causal diagonal for this row.
__device__ __forceinline__ void mask32(float (&s)[32], int lo, int lim) {
#pragma unroll
    for (int i = 0; i < 32; ++i)
        if (i >= lim || i < lo) s[i] = -INFINITY;
}
// p = 2^(s*c - m) for 32 keys -> 16 packed bf16 pairs; row sums into four accumulators.  With kPoly,
// kPolyOf4 of every four pairs take the FMA-pipe polynomial instead of MUFU; masked tiles do not (the
// polynomial clamps a masked score, -inf, to 2^-126, which is not the exact zero a hidden key needs).
template <bool kPoly>
__device__ __forceinline__ void exp32(const float (&s)[32], uint32_t (&pk)[16], float2 c2, float2 nm2, float2& sum0,
                                      float2& sum1, float2& sum2, float2& sum3) {
#pragma unroll
    for (int i = 0; i < 16; i += 4) {
        const float2 x0 = __ffma2_rn(make_float2(s[2 * i + 0], s[2 * i + 1]), c2, nm2);
        const float2 x1 = __ffma2_rn(make_float2(s[2 * i + 2], s[2 * i + 3]), c2, nm2);
        const float2 x2 = __ffma2_rn(make_float2(s[2 * i + 4], s[2 * i + 5]), c2, nm2);
        const float2 x3 = __ffma2_rn(make_float2(s[2 * i + 6], s[2 * i + 7]), c2, nm2);
        const float2 p0 = make_float2(ex2(x0.x), ex2(x0.y));
        const float2 p1 = make_float2(ex2(x1.x), ex2(x1.y));
        const float2 p2 = (kPoly && kPolyOf4 >= 2) ? ex2_poly2(x2) : make_float2(ex2(x2.x), ex2(x2.y));
        const float2 p3 = (kPoly && kPolyOf4 >= 1) ? ex2_poly2(x3) : make_float2(ex2(x3.x), ex2(x3.y));
        sum0 = __fadd2_rn(sum0, p0);
        sum1 = __fadd2_rn(sum1, p1);
        sum2 = __fadd2_rn(sum2, p2);
        sum3 = __fadd2_rn(sum3, p3);
        pk[i + 0] = pack_bf16(p0.x, p0.y);
        pk[i + 1] = pack_bf16(p1.x, p1.y);
        pk[i + 2] = pack_bf16(p2.x, p2.y);
        pk[i + 3] = pack_bf16(p3.x, p3.y);
    }
}

// The same for the FP8 variant: 32 weights -> 8 TMEM columns of four E4M3 bytes each (the caller's exponent
// offset already holds the 2^kP8Shift scaling); the row sums take the unrounded values.
__device__ __forceinline__ void exp32_f8(const float (&s)[32], uint32_t (&pk)[8], float2 c2, float2 nm2, float2& sum0,
                                         float2& sum1, float2& sum2, float2& sum3) {
#pragma unroll
    for (int i = 0; i < 8; i += 2) {
        const float2 x0 = __ffma2_rn(make_float2(s[4 * i + 0], s[4 * i + 1]), c2, nm2);
        const float2 x1 = __ffma2_rn(make_float2(s[4 * i + 2], s[4 * i + 3]), c2, nm2);
        const float2 x2 = __ffma2_rn(make_float2(s[4 * i + 4], s[4 * i + 5]), c2, nm2);
        const float2 x3 = __ffma2_rn(make_float2(s[4 * i + 6], s[4 * i + 7]), c2, nm2);
        const float2 p0 = make_float2(ex2(x0.x), ex2(x0.y));
        const float2 p1 = make_float2(ex2(x1.x), ex2(x1.y));
        const float2 p2 = make_float2(ex2(x2.x), ex2(x2.y));
        const float2 p3 = make_float2(ex2(x3.x), ex2(x3.y));
        sum0 = __fadd2_rn(sum0, p0);
        sum1 = __fadd2_rn(sum1, p1);
        sum2 = __fadd2_rn(sum2, p2);
        sum3 = __fadd2_rn(sum3, p3);
        pk[i + 0] = pack_e4m3x4(p0.x, p0.y, p1.x, p1.y);
        pk[i + 1] = pack_e4m3x4(p2.x, p2.y, p3.x, p3.y);
    }
}

struct SoftmaxSync {
    uint32_t bars;                   // shared-memory address of the barrier array
    uint32_t s_ready_id;             // barrier "a score tile of this head is in the S buffer"
    uint32_t pv_done_id, pv_parity;  // barrier and phase of this head's previous P*V
    volatile uint32_t* abort_flag;
    int32_t* status;
    int iter;
};

// Reads the 128 scores of this thread's row from the S buffer (the caller has seen s_ready).
#define CP_LOAD_S(a0, a1, a2, a3)          \
    TMEM_LD32(s_tmem + 0, a0, 0);          \
    TMEM_LD32(s_tmem + 32, a1, 0);         \
    TMEM_LD32(s_tmem + 64, a2, 0);         \
    TMEM_LD32(s_tmem + 96, a3, 0);

// Hands the S buffer back once this warp's loads have landed: one arrival per warp.
__device__ __forceinline__ void release_s(uint32_t bars) {
    tc_wait_ld();
    tc_fence_before();
    __syncwarp();
    if ((threadIdx.x & 31) == 0) mbar_arrive(bars + kBarSFree * 8);
}

// One 128x128 score tile of one head; the row's scores are already in registers (c0..c3).  Row max, lazy
// rescale, exponentials in four pieces of 32 keys, P into this head's TMEM columns piece by piece (the P*V
// issuer is signalled after the third piece and after the last).  If the head has another tile in this
// unit, its scores replace the current ones before the function returns: the first 96 columns already
// after the third piece when the tile is in the S buffer by then (their registers are no longer needed,
// so the load runs under the last exponentials), the rest -- or all of it, after a wait -- behind the
// last piece.  The S buffer goes back to the score issuer as soon as the loads have landed.
// Straight-line code in both variants, no per-element branches.
// kMasked: some keys of the tile are hidden from some rows (causal diagonal, or the edge of the unit's key
// range); this row sees columns [lo, lim).
template <bool kMasked, bool kFp8>
__device__ __forceinline__ void softmax_tile(float (&c0)[32], float (&c1)[32], float (&c2)[32], float (&c3)[32],
                                             bool more, uint32_t& s_par, uint32_t s_tmem, uint32_t p_tmem,
                                             uint32_t o_tmem, uint32_t p_bar0, float c, int lo, int lim, bool first,
                                             float& m, float& l, const SoftmaxSync& sy) {
    if (kMasked) {
        mask32(c0, lo, lim);
        mask32(c1, lo - 32, lim - 32);
        mask32(c2, lo - 64, lim - 64);
        mask32(c3, lo - 96, lim - 96);
    }
    float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
    max32(c0, mx0, mx1, mx2, mx3);
    max32(c1, mx0, mx1, mx2, mx3);
    max32(c2, mx0, mx1, mx2, mx3);
    max32(c3, mx0, mx1, mx2, mx3);
    const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3));
    const float m_new = fmaxf(m, mx * c);
    if (first) {
        m = m_new;     // O is overwritten by the first P*V: nothing to rescale
    } else {
        // P and O of this head are free once the previous tile's P*V has finished (long ago, normally)
        mbar_wait(sy.bars, sy.pv_done_id, sy.pv_parity, sy.abort_flag, sy.status, sy.iter);
        __syncwarp();
        tc_fence_after();
        const bool grow = (m_new - m) > (kFp8 ? kRescaleThreshold8 : kRescaleThreshold);
        if (__any_sync(0xffffffffu, grow)) {
            const float m_upd = grow ? m_new : m;
            const float alpha = ex2(m - m_upd);
            l *= alpha;
            m = m_upd;
#pragma unroll 1
            for (int cc = 0; cc < 4; ++cc) {
                float o[32];
                TMEM_LD32(o_tmem + cc * 32, o, 0);
                tc_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] *= alpha;
                TMEM_ST32F(o_tmem + cc * 32, o, 0);
            }
        }
    }
    const float2 c2f = make_float2(c, c);
    // a row that has seen no key yet (only possible in masked tiles of a KV-split piece) keeps m = -inf;
    // subtracting 0 instead keeps its weights at exactly 0 rather than NaN
    const float m_sub = ((kMasked && m == -INFINITY) ? 0.f : m) - (kFp8 ? kP8Shift : 0.f);
    const float2 nm2 = make_float2(-m_sub, -m_sub);
    float2 sum0 = make_float2(0.f, 0.f), sum1 = sum0, sum2 = sum0, sum3 = sum0;
    uint32_t pk[kFp8 ? 8 : 16];
#define CP_P_PIECE(cur, q)                                                              \
    if constexpr (kFp8) {                                                               \
        exp32_f8(cur, pk, c2f, nm2, sum0, sum1, sum2, sum3);                            \
        TMEM_ST8R(p_tmem + (q) * 8, pk, 0);                                             \
    } else {                                                                            \
        exp32<!kMasked>(cur, pk, c2f, nm2, sum0, sum1, sum2, sum3);                     \
        TMEM_ST16R(p_tmem + (q) * 16, pk, 0);                                           \
    }                                                                                   \
    if ((q) + 1 == kSplitQ || (q) == 3) {                                               \
        tc_wait_st();                                                                   \
        tc_fence_before();                                                              \
        __syncwarp();                                                                   \
        if ((threadIdx.x & 31) == 0) mbar_arrive(p_bar0 + ((q) == 3 ? 1 : 0) * 8);      \
    }
    CP_P_PIECE(c0, 0)
    CP_P_PIECE(c1, 1)
    CP_P_PIECE(c2, 2)
    // is the head's next score tile in the S buffer already?  (same answer in the whole warp)
    bool early = false;
    if (more) {
        early = __all_sync(0xffffffffu, mbar_test(sy.bars + sy.s_ready_id * 8, s_par));
        if (early) {
            tc_fence_after();
            TMEM_LD32(s_tmem + 0, c0, 0);
            TMEM_LD32(s_tmem + 32, c1, 0);
            TMEM_LD32(s_tmem + 64, c2, 0);
        }
    }
    CP_P_PIECE(c3, 3)
#undef CP_P_PIECE
    if (more) {
        if (!early) {
            mbar_wait(sy.bars, sy.s_ready_id, s_par, sy.abort_flag, sy.status, sy.iter);
            __syncwarp();
            tc_fence_after();
            TMEM_LD32(s_tmem + 0, c0, 0);
            TMEM_LD32(s_tmem + 32, c1, 0);
            TMEM_LD32(s_tmem + 64, c2, 0);
        }
        TMEM_LD32(s_tmem + 96, c3, 0);
        release_s(sy.bars);
        s_par ^= 1u;
    }
    const float2 st = __fadd2_rn(__fadd2_rn(sum0, sum1), __fadd2_rn(sum2, sum3));
    l += st.x + st.y;
}

// 4 x 4 transpose of 16-byte items inside every group of four lanes: on return v[s] holds what lane (quad * 4 + s)
// had in v[t], t = this lane's position in its quad.  Two exchange stages (lane ^ 1, lane ^ 2), 16 shuffles.
__device__ __forceinline__ uint4 shfl_xor16(uint4 a, int mask) {
    a.x = __shfl_xor_sync(0xffffffffu, a.x, mask);
    a.y = __shfl_xor_sync(0xffffffffu, a.y, mask);
    a.z = __shfl_xor_sync(0xffffffffu, a.z, mask);
    a.w = __shfl_xor_sync(0xffffffffu, a.w, mask);
    return a;
}
__device__ __forceinline__ void quad_transpose(uint4 (&v)[4], int t) {
    {
        const bool hi = t & 1;
        const uint4 r0 = shfl_xor16(hi ? v[0] : v[1], 1), r1 = shfl_xor16(hi ? v[2] : v[3], 1);
        if (hi) { v[0] = r0; v[2] = r1; } else { v[1] = r0; v[3] = r1; }
    }
    {
        const bool hi = t & 2;
        const uint4 r0 = shfl_xor16(hi ? v[0] : v[2], 2), r1 = shfl_xor16(hi ? v[1] : v[3], 2);
        if (hi) { v[0] = r0; v[1] = r1; } else { v[2] = r0; v[3] = r1; }
    }
}

template <bool kFp8>
__device__ __forceinline__ void softmax_role(const AttnParams& p, const InlineSched& inl, uint32_t smem_base, uint32_t tmem_base,
                                             volatile uint32_t* abort_flag, int wg) {
    const uint32_t bars = smem_base + kSmemBar;
    const int lane = threadIdx.x & 31;
    const int warp_in_wg = (threadIdx.x >> 5) & 3;
    const uint32_t lane_addr = (uint32_t)(warp_in_wg * 32) << 16;   // TMEM lane field of this warp
    const uint32_t s_tmem = tmem_base + lane_addr + kTmemS;
    const uint32_t p_tmem = tmem_base + lane_addr + kTmemP + wg * 64;
    const uint32_t o_tmem = tmem_base + lane_addr + kTmemO + wg * 128;
    const uint32_t p_bar0 = bars + (kBarPReady + wg * 4) * 8;
    // this thread's query row inside the unit: TMEM lane, plus 128 for the second tile of a tile-pair unit;
    // its head: head wg of the pair, or the unit's only head
    const bool tile_pair = p.heads_per_unit == 1;
    const int row = warp_in_wg * 32 + lane + (tile_pair ? wg * kBlockM : 0);
    const int head_sel = tile_pair ? 0 : wg;
    const int row_base = tile_pair ? wg * kBlockM : 0;              // first row of this warpgroup's tile in the unit
    float c = p.scale_log2;
    uint32_t tile_cnt = 0;

#define SM_WAIT(id, parity, it)                                                                  \
    mbar_wait(bars, (id), (parity), abort_flag, p.status, (it));                                 \
    __syncwarp();
    uint32_t s_par = 0;        // phase parity of s_ready for this head

    UnitInfo u, nu;
    bool have = fetch_unit(p, inl, 0, u);
    for (int round = 0; have; ++round) {
        const int n = u.t_end;
        const int head = u.head0 + head_sel;
        const int j_first = u.t_begin;
        float m = -INFINITY;   // running row max in log2 units (possibly stale by < threshold)
        float l = 0.f;         // running row sum of 2^(s - m)
        if (kFp8)              // raw scores are products of codes: this row's query scale and the head's key scale
            c = p.scale_log2 * p.k_scale[u.kv_head] *
                (row < u.it.n_rows ? p.q_scale[((int64_t)u.it.q_row0 + row) * p.Hq + head] : 0.f);
        // tiles below n_full lie entirely under the causal diagonal of every row of this warpgroup's q-tile and
        // inside the unit's key range; the range's first tile is cut on the left when kv_lo is not a tile
        // multiple.  (The earlier tile of a tile-pair unit finds the unit's last KV tile fully masked.)
        const int n_full = min(u.it.kv_len0 + row_base, u.it.kv_hi) / kBlockN;
        const int j_cut = (u.it.kv_lo & (kBlockN - 1)) ? (u.it.kv_lo >> 7) : -1;
        float s0[32], s1[32], s2[32], s3[32];   // the row's scores of the current tile
        // the first tile of the unit is loaded here, every later one by the tile before it
        SM_WAIT(kBarSReady + wg, s_par, j_first);
        s_par ^= 1u;
        tc_fence_after();
        CP_LOAD_S(s0, s1, s2, s3)
        release_s(bars);
#pragma unroll 1
        for (int j = j_first; j < n; ++j) {
            const SoftmaxSync sy = {bars, kBarSReady + (uint32_t)wg, kBarPvDone + (uint32_t)wg, (tile_cnt - 1) & 1,
                                    abort_flag, p.status, j};
            if (j < n_full && j != j_cut)
                softmax_tile<false, kFp8>(s0, s1, s2, s3, j + 1 < n, s_par, s_tmem, p_tmem, o_tmem, p_bar0, c, 0, 0,
                                          j == j_first, m, l, sy);
            else
                softmax_tile<true, kFp8>(s0, s1, s2, s3, j + 1 < n, s_par, s_tmem, p_tmem, o_tmem, p_bar0, c,
                                   u.it.kv_lo - j * kBlockN, min(u.it.kv_len0 + row, u.it.kv_hi) - j * kBlockN,
                                   j == j_first, m, l, sy);
            ++tile_cnt;
        }
        // the next unit's description is fetched under the epilogue
        const bool have_next = fetch_unit(p, inl, round + 1, nu);
        // epilogue: O / l -> global at the row's original position; LSE in natural log
        SM_WAIT(kBarPvDone + wg, (tile_cnt - 1) & 1, n);
        tc_fence_after();
        // a row of a KV-split piece may see none of the piece's keys: l = 0, written as O = 0, lse = -inf
        // (FP8 variant: O and l both carry the 2^kP8Shift factor of the weights, which cancels; V's scale joins here)
        const float inv_l = (l > 0.f) ? (kFp8 ? p.v_scale[u.kv_head] : 1.f) / l : 0.f;
        const bool partial = u.slot >= 0;
        const bool valid = row < u.it.n_rows;
        const int64_t grow_idx = (int64_t)u.it.q_row0 + row;
        // A thread holds 32 consecutive columns of its own row; written as they are, every store instruction of a warp
        // would touch 32 rows with 16 bytes each.  The four lanes of a quad swap their 16-byte pieces first, so that
        // a store instruction writes 64 contiguous bytes of each of 8 rows (a quarter of the memory transactions).
        const int qt = lane & 3;
        const int row_q0 = row - qt;                                        // first row of this lane's quad
        const bool f32 = partial || p.out_f32;
        // element (not byte) offset of row row_q0, column 0, in the destination this call writes
        const int64_t base_q0 = partial ? (((int64_t)u.slot * 2 + wg) * kBlockM + (row_q0 - row_base)) * kD
                                        : (((int64_t)u.it.q_row0 + row_q0) * p.Hq + head) * kD;
        const int64_t row_pitch = partial ? kD : (int64_t)p.Hq * kD;        // elements between consecutive rows
#pragma unroll 1
        for (int cc = 0; cc < 4; ++cc) {
            float o[32];
            TMEM_LD32(o_tmem + cc * 32, o, 0);
            tc_wait_ld();
            if (f32) {
                float* dstf = partial ? p.partial_o : reinterpret_cast<float*>(p.out);
#pragma unroll
                for (int hlf = 0; hlf < 2; ++hlf) {
                    uint4 v[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int c0 = hlf * 16 + 4 * i;
                        v[i] = make_uint4(__float_as_uint(o[c0] * inv_l), __float_as_uint(o[c0 + 1] * inv_l),
                                          __float_as_uint(o[c0 + 2] * inv_l), __float_as_uint(o[c0 + 3] * inv_l));
                    }
                    quad_transpose(v, qt);
#pragma unroll
                    for (int sdx = 0; sdx < 4; ++sdx)
                        if (row_q0 + sdx < u.it.n_rows)
                            *reinterpret_cast<uint4*>(dstf + base_q0 + sdx * row_pitch + cc * 32 + hlf * 16 + qt * 4) = v[sdx];
                }
            } else {
                uint4 v[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    v[i].x = pack_bf16(o[8 * i + 0] * inv_l, o[8 * i + 1] * inv_l);
                    v[i].y = pack_bf16(o[8 * i + 2] * inv_l, o[8 * i + 3] * inv_l);
                    v[i].z = pack_bf16(o[8 * i + 4] * inv_l, o[8 * i + 5] * inv_l);
                    v[i].w = pack_bf16(o[8 * i + 6] * inv_l, o[8 * i + 7] * inv_l);
                }
                quad_transpose(v, qt);
                __nv_bfloat16* dsth = reinterpret_cast<__nv_bfloat16*>(p.out);
#pragma unroll
                for (int sdx = 0; sdx < 4; ++sdx)
                    if (row_q0 + sdx < u.it.n_rows)
                        *reinterpret_cast<uint4*>(dsth + base_q0 + sdx * row_pitch + cc * 32 + qt * 8) = v[sdx];
            }
        }
        if (valid) {
            const float lse_val = (l > 0.f) ? (m + lg2(l) - (kFp8 ? kP8Shift : 0.f)) * 0.6931471805599453f : -INFINITY;
            if (partial) p.partial_lse[((int64_t)u.slot * 2 + wg) * kBlockM + (row - row_base)] = lse_val;
            else p.lse[(int64_t)head * p.lse_stride + grow_idx] = lse_val;
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bars + (kBarOFree + wg) * 8);
        u = nu;
        have = have_next;
    }
#undef SM_WAIT
}

// The spare warp of every CTA: rows of a partial-result call that no tile covers (rows of other shards, rows
// that see no key of the key range) get zeros and lse = -inf here, so that the call needs no launch besides
// this one.  out is fp32 [rows, Hq, D], so a row range is one contiguous run of floats.
__device__ __forceinline__ void fill_role(const AttnParams& p) {
    const int lane = threadIdx.x & 31;
    const int64_t start = (int64_t)blockIdx.x * 32 + lane, stride = (int64_t)gridDim.x * 32;
    for (int g = 0; g < p.n_fill; ++g) {
        const int64_t b = p.fill[2 * g], n = p.fill[2 * g + 1] - b;
        float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + b * p.Hq * kD);
        const int64_t n4 = n * p.Hq * (kD / 4);
        for (int64_t i = start; i < n4; i += stride) o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
        const int64_t nl = n * p.Hq;
        for (int64_t i = start; i < nl; i += stride) {
            const int64_t h = i / n;
            p.lse[h * p.lse_stride + b + (i - h * n)] = -INFINITY;
        }
    }
}

// kFp8: the FP8 K/V variant (one-byte Q / K / V / P operands).
template <bool kFp8>
__global__ void __launch_bounds__(kThreads, 1)
cp_attn_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const AttnParams p, const __grid_constant__ InlineSched inl) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* smem_gen = smem_raw + (smem_base - smem_u32(smem_raw));
    volatile uint32_t* tmem_ptr = reinterpret_cast<volatile uint32_t*>(smem_gen + kSmemTmemPtr);
    volatile uint32_t* abort_flag = reinterpret_cast<volatile uint32_t*>(smem_gen + kSmemAbort);
    const int warp = threadIdx.x >> 5;
    const uint32_t bars = smem_base + kSmemBar;

    if (threadIdx.x == 0) {
        mbar_init(bars + kBarQFull * 8, 1);
        mbar_init(bars + kBarQEmpty * 8, 1);
        for (int s = 0; s < kKvStages; ++s) {
            mbar_init(bars + (kBarKvFull + s) * 8, 1);
            mbar_init(bars + (kBarKvEmpty + s) * 8, 1);
        }
        mbar_init(bars + kBarSFree * 8, 4);
        for (int w = 0; w < 2; ++w) {
            mbar_init(bars + (kBarSReady + w) * 8, 1);
            for (int q4 = 0; q4 < 4; ++q4) mbar_init(bars + (kBarPReady + 4 * w + q4) * 8, 4);   // one arrival per warp
            mbar_init(bars + (kBarPvDone + w) * 8, 1);
            mbar_init(bars + (kBarOFree + w) * 8, 4);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_base + kSmemTmemPtr), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_ptr;

    if (warp < 8) {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        softmax_role<kFp8>(p, inl, smem_base, tmem_base, abort_flag, warp >> 2);
    } else {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsOther));
        if (warp == 8) {
            producer_role<kFp8>(&tmQ, &tmK, &tmV, p, inl, smem_base, abort_flag, 0, p.co_producer ? 1 : 2);
        } else if (warp == 9) {
            mma_s_role<kFp8>(p, inl, smem_base, tmem_base, abort_flag);
        } else if (warp == 10) {
            mma_pv_role<kFp8>(p, inl, smem_base, tmem_base, abort_flag);
        } else if (p.n_fill > 0) {
            fill_role(p);
        } else if (!kFp8 && p.co_producer) {
            producer_role<kFp8>(&tmQ, &tmK, &tmV, p, inl, smem_base, abort_flag, 1, 2);
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // give copies that are still in flight time to land before shared memory is released
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 0) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// Self-test of the bounded wait: one warp waits on a barrier that nothing ever arrives at, with a short
// limit.  The wait gives up, records CP_ERR_TIMEOUT in the status words and the kernel returns.
__global__ void wait_expiry_selftest_kernel(int32_t* status, long long limit_cycles) {
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    mbar_wait(smem_u32(&bar), 0, 0, &abort_flag, status, 7, limit_cycles);
}

// Rows [b, b + n) of a partial result that the call computes nothing for: zeros and lse = -inf.  Only used when
// the attention kernel itself is not launched (the shard owns no row) or has more gaps than it takes.
__global__ void fill_rows_kernel(float* out, float* lse, int64_t lse_stride, int64_t b, int64_t n, int Hq) {
    const int64_t start = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, stride = (int64_t)gridDim.x * blockDim.x;
    float4* o = reinterpret_cast<float4*>(out + b * Hq * kD);
    const int64_t n4 = n * Hq * (kD / 4);
    for (int64_t i = start; i < n4; i += stride) o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    const int64_t nl = n * Hq;
    for (int64_t i = start; i < nl; i += stride) {
        const int64_t h = i / n;
        lse[h * lse_stride + b + (i - h * n)] = -INFINITY;
    }
}

// LSE merge of the KV-split units: block b combines the partial slots of merges[b] into the final
// rows.  One warp per (head, row), one float4 per lane; weights exp(lse_k - max) by fast exp.
struct FixupParams {
    const TileItem* items;
    const MergeEntry* merges;
    const int32_t* merge_slots;
    const float* partial_o;
    const float* partial_lse;
    void* out;
    int32_t out_f32;
    int32_t Hq;
    int32_t heads_per_unit;
    float* lse;
    int64_t lse_stride;
    int32_t inl_items, inl_merges, inl_merge_slots;   // >= 0: the list sits at this byte offset of the launch-parameter copy
};

constexpr int kFixupRowsPerBlock = 8;     // one (head, row) combination per warp

// grid = (split units, 256 / kFixupRowsPerBlock): each warp combines one row.  The partial LSEs of the row are
// loaded 32 slots at a time (lane k holds slot k), max and sum by warp shuffles; units cut into at most 32 pieces
// (all but pathological schedules) read every LSE once.  The partial rows are fetched four at a time, all loads
// issued before the first use.
__global__ void __launch_bounds__(256) cp_attn_fixup_kernel(const FixupParams p, const __grid_constant__ InlineSched inl) {
    const TileItem* items = p.inl_items >= 0 ? reinterpret_cast<const TileItem*>(inl.bytes + p.inl_items) : p.items;
    const MergeEntry* merges = p.inl_merges >= 0 ? reinterpret_cast<const MergeEntry*>(inl.bytes + p.inl_merges) : p.merges;
    const int32_t* merge_slots = p.inl_merge_slots >= 0 ? reinterpret_cast<const int32_t*>(inl.bytes + p.inl_merge_slots) : p.merge_slots;
    const MergeEntry me = merges[blockIdx.x];
    const TileItem it = items[me.item];
    const int lane = threadIdx.x & 31;
    const int warp = threadIdx.x >> 5;
    const int hr = blockIdx.y * kFixupRowsPerBlock + warp;
    const int wg = hr / kBlockM;                  // head wg of the pair, or (tile-pair unit) rows 128 wg .. of the one head
    const int row = hr - wg * kBlockM;
    const int urow = p.heads_per_unit == 2 ? row : hr;     // row inside the unit
    if (urow >= it.n_rows) return;
    // pass 1: max of the partial LSEs (lane k of each group of 32 slots holds slot k)
    float m = -INFINITY;
    int slot0 = 0;
    float lse0 = -INFINITY;        // the first group's values stay in registers for pass 2
    for (int base = 0; base < me.n_slots; base += 32) {
        if (base + lane < me.n_slots) {
            const int slot = merge_slots[me.slot_off + base + lane];
            const float v = p.partial_lse[((int64_t)slot * 2 + wg) * kBlockM + row];
            if (base == 0) { slot0 = slot; lse0 = v; }
            m = fmaxf(m, v);
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    // pass 2: weights exp(lse_k - m) and the weighted sum of the partial rows
    float wsum = 0.f;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int base = 0; base < me.n_slots; base += 32) {
        int my_slot = slot0;
        float my_lse = lse0;
        if (base > 0) {
            my_lse = -INFINITY;
            if (base + lane < me.n_slots) {
                my_slot = merge_slots[me.slot_off + base + lane];
                my_lse = p.partial_lse[((int64_t)my_slot * 2 + wg) * kBlockM + row];
            }
        }
        const float w_mine = (my_lse == -INFINITY) ? 0.f : __expf(my_lse - m);
        wsum += w_mine;
        const int cnt = min(32, me.n_slots - base);
        for (int k0 = 0; k0 < cnt; k0 += 4) {
            float w[4];
            float4 x[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                // lanes beyond the group hold weight 0; their slot index (0 or a real one) is a valid slot to read
                w[k] = __shfl_sync(0xffffffffu, w_mine, (k0 + k) & 31);
                const int slot = __shfl_sync(0xffffffffu, my_slot, (k0 + k) & 31);
                x[k] = (k0 + k < cnt && w[k] > 0.f)
                           ? reinterpret_cast<const float4*>(p.partial_o + (((int64_t)slot * 2 + wg) * kBlockM + row) * kD)[lane]
                           : make_float4(0.f, 0.f, 0.f, 0.f);     // a zero weight hides whatever the slot holds for this row
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float wk = (k0 + k < cnt) ? w[k] : 0.f;
                acc.x = fmaf(wk, x[k].x, acc.x);
                acc.y = fmaf(wk, x[k].y, acc.y);
                acc.z = fmaf(wk, x[k].z, acc.z);
                acc.w = fmaf(wk, x[k].w, acc.w);
            }
        }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
    // a row may see none of the unit's keys (a key range that starts behind its causal limit): zeros, -inf
    const float inv = wsum > 0.f ? 1.f / wsum : 0.f;
    const int head = p.heads_per_unit == 2 ? 2 * me.pair + wg : me.pair;
    const int64_t grow = (int64_t)it.q_row0 + urow;
    const int64_t off = (grow * p.Hq + head) * kD + lane * 4;
    if (p.out_f32) {
        *reinterpret_cast<float4*>(reinterpret_cast<float*>(p.out) + off) =
            make_float4(acc.x * inv, acc.y * inv, acc.z * inv, acc.w * inv);
    } else {
        uint2 pk;
        pk.x = pack_bf16(acc.x * inv, acc.y * inv);
        pk.y = pack_bf16(acc.z * inv, acc.w * inv);
        *reinterpret_cast<uint2*>(reinterpret_cast<__nv_bfloat16*>(p.out) + off) = pk;
    }
    if (lane == 0) p.lse[(int64_t)head * p.lse_stride + grow] = wsum > 0.f ? m + __logf(wsum) : -INFINITY;
}

}  // namespace

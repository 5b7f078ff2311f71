// bf16 tree attention for sm_100a: split-KV flash-decoding with TMA-staged K/V tiles and tcgen05
// MMAs accumulating in tensor memory (Section 4.4: every tree row attends to the cached prefix
// and, inside the tree, to the rows named by its ancestor mask).
//
// Rows of one KV head are the (node, g) pairs of its G = Hq/Hkv query heads, row = node*G + g, so
// that budget x G rows share each K/V tile and QK^T / PV are dense 128x128x128 contractions.
//
// One CTA = one (request, KV head, 128-row tile, KV split).  Warp roles:
//   warps 0-7  softmax: two threads per row (TMEM lane = row).  Thread (row, h) owns key columns
//              [64h, 64h+64) of every KV tile with its OWN reference maximum, sum and O accumulator
//              (O_0, O_1 in TMEM), so the halves of a row never synchronise inside the loop; at the end
//              they are merged like two KV splits.  Exponentials (MUFU) are the co-bottleneck of this
//              kernel, so all eight warps work on every tile
//   warp 8     TMA producer: Q once, then separate 3-stage rings for K tiles and V tiles
//   warp 9     MMA issuer: S = Q K^T (operands in shared memory) runs one tile ahead into two TMEM
//              score buffers; O_h += P_h V_h (P read from TMEM, V as an MN-major shared-memory
//              operand) as soon as half h of the tile is ready; owns the TMEM allocation
// A last row tile of at most 16 rows (the root's G rows of a tree of 2^k nodes) takes a path of its own
// in batches that fill the SMs several times over: see tail_tile_cta.
// The ancestor bitmask is applied only on tree tiles; prefix tiles need at most a length test on
// the request's last tile.  Each split writes its normalised rows (fp16) with their reference maximum
// and sum; a combine kernel merges them by log-sum-exp.  Every wait is bounded: when one gives up, the CTA raises a flag in the
// device status word, drains its copies and leaves without touching its outputs.
#include "common.cuh"
#include <cuda.h>
#include <cuda_fp16.h>
#include <math_constants.h>
#include <algorithm>
#include <mutex>
#include <unordered_map>
#include <vector>

namespace ddtree {
namespace {

constexpr int kTile = 128;            // rows per CTA, keys per KV tile, head dim
constexpr int kStages = 3;
constexpr int kSBufs = 2;              // score buffers in TMEM: Q K^T runs one tile ahead of the softmax
constexpr int kSoftmaxThreads = 256;   // two threads per row, 64 key columns each
constexpr int kGroupThreads = 128;     // threads of one column half
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr int kThreads = 320;          // warps 0-7: softmax; 8: TMA producer; 9: MMA issuer
constexpr uint32_t kHalfBytes = 128 * 64 * 2;      // one 64-wide half of a 128x128 bf16 tile
constexpr uint32_t kTileBytes = 2 * kHalfBytes;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;         // S buffers at columns 0 and 128; half h's bf16 P overwrites columns [64h, 64h+32)
constexpr uint32_t kColO = 256;       // O accumulators of the two column halves at columns 256 and 384
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2e = 1.4426950408889634f;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kMaxOrdered = 128;
constexpr uint32_t kErrTimeout = 0x5101;
constexpr uint32_t kErrAlign = 0x5102;

// ---- PTX wrappers --------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Non-blocking test of a phase.  try_wait may park the thread for a while and costs a couple of
// hundred cycles even when the phase has long completed; test_wait answers at once, so every wait
// starts with it and several barriers can be tested back to back.
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.b32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait.  Returns false when it gave up (or another thread of the CTA already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
    if (mbar_test(bar, parity)) return true;
    for (uint32_t i = 0; i < kSpinLimit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) {
            __nanosleep(64);
            if ((i & 255u) == 0 && *abort_flag) return false;
        }
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1, int c2, int c3) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1), "r"(c2), "r"(c3) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// One lane of a converged warp (all 32 lanes must call this together).
__device__ __forceinline__ bool elect_one() {
    uint32_t pred;
    asm volatile(
        "{\n\t.reg .pred P1;\n\t.reg .b32 r;\n\t"
        "elect.sync r|P1, 0xffffffff;\n\t"
        "selp.b32 %0, 1, 0, P1;\n\t}"
        : "=r"(pred));
    return pred != 0;
}
// D[tmem] (+)= A[smem desc] * B[smem desc].  The accumulate flag is a template argument and the
// operands are "base + constant": one thread issues every MMA of the CTA, and anything beyond a
// handful of scalar instructions per MMA makes that thread, not the tensor pipe, the bottleneck.
template <bool kAccumulate>
__device__ __forceinline__ void umma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc) {
    if (kAccumulate)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                     ::"r"(d), "l"(a), "l"(b), "r"(idesc) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
template <bool kAccumulate>
__device__ __forceinline__ void umma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc) {
    if (kAccumulate)
        asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                     ::"r"(d), "r"(a), "l"(b), "r"(idesc) : "memory");
    else
        asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\t"
                     "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                     ::"r"(d), "r"(a), "l"(b), "r"(idesc) : "memory");
}

#define DDTREE_R32(a, o) \
    "=r"(a[o + 0]), "=r"(a[o + 1]), "=r"(a[o + 2]), "=r"(a[o + 3]), "=r"(a[o + 4]), "=r"(a[o + 5]), "=r"(a[o + 6]),     \
    "=r"(a[o + 7]), "=r"(a[o + 8]), "=r"(a[o + 9]), "=r"(a[o + 10]), "=r"(a[o + 11]), "=r"(a[o + 12]), "=r"(a[o + 13]), \
    "=r"(a[o + 14]), "=r"(a[o + 15]), "=r"(a[o + 16]), "=r"(a[o + 17]), "=r"(a[o + 18]), "=r"(a[o + 19]),               \
    "=r"(a[o + 20]), "=r"(a[o + 21]), "=r"(a[o + 22]), "=r"(a[o + 23]), "=r"(a[o + 24]), "=r"(a[o + 25]),               \
    "=r"(a[o + 26]), "=r"(a[o + 27]), "=r"(a[o + 28]), "=r"(a[o + 29]), "=r"(a[o + 30]), "=r"(a[o + 31])
#define DDTREE_W32(a, o) \
    "r"(a[o + 0]), "r"(a[o + 1]), "r"(a[o + 2]), "r"(a[o + 3]), "r"(a[o + 4]), "r"(a[o + 5]), "r"(a[o + 6]),     \
    "r"(a[o + 7]), "r"(a[o + 8]), "r"(a[o + 9]), "r"(a[o + 10]), "r"(a[o + 11]), "r"(a[o + 12]), "r"(a[o + 13]), \
    "r"(a[o + 14]), "r"(a[o + 15]), "r"(a[o + 16]), "r"(a[o + 17]), "r"(a[o + 18]), "r"(a[o + 19]),             \
    "r"(a[o + 20]), "r"(a[o + 21]), "r"(a[o + 22]), "r"(a[o + 23]), "r"(a[o + 24]), "r"(a[o + 25]),             \
    "r"(a[o + 26]), "r"(a[o + 27]), "r"(a[o + 28]), "r"(a[o + 29]), "r"(a[o + 30]), "r"(a[o + 31])
#define DDTREE_L32 \
    "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "   \
    "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}"
#define DDTREE_S32 \
    "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "  \
    "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32}"

// 32 consecutive columns of this thread's TMEM lane -> v[o .. o+31]
#define TMEM_LD32(v, o, taddr) \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 " DDTREE_L32 ", [%32];" : DDTREE_R32(v, o) : "r"(taddr))
#define TMEM_ST32(taddr, v, o) \
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], " DDTREE_S32 ";" ::"r"(taddr), DDTREE_W32(v, o) : "memory")
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// 16 consecutive columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld16(uint32_t (&v)[16], uint32_t taddr) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr));
}
// Named barriers of the short-tile path: id 1 + g over the 128 threads of key group g (plain and with an
// OR vote), id 3 over both groups.
__device__ __forceinline__ void bar_keys(int g) { asm volatile("bar.sync %0, 128;" ::"r"(1 + g) : "memory"); }
__device__ __forceinline__ bool bar_keys_or(int g, bool x) {
    uint32_t r;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.b32 q, %2, 0;\n\tbar.red.or.pred p, %1, 128, q;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(r) : "r"(1 + g), "r"(static_cast<uint32_t>(x)) : "memory");
    return r != 0;
}
__device__ __forceinline__ void bar_all_keys() { asm volatile("bar.sync 3, 256;" ::: "memory"); }

// Shared-memory matrix descriptor: 128-byte swizzle, 8-row groups 1024 bytes apart.
//   K-major operand (Q, K): rows of 64 bf16 (128 bytes); the leading-dimension field is unused.
//   MN-major operand (V):   rows are keys (the contraction index), 64 head-dim elements per row;
//                           `lbo_bytes` is the distance between the two 64-wide head-dim halves.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes) {
    uint64_t d = 0;
    d |= static_cast<uint64_t>((addr & 0x3ffffu) >> 4);
    d |= static_cast<uint64_t>((lbo_bytes >> 4) & 0x3fffu) << 16;
    d |= static_cast<uint64_t>(1024u >> 4) << 32;
    d |= 1ull << 46;  // descriptor version of this architecture
    d |= 2ull << 61;  // 128-byte swizzle
    return d;
}
// Instruction descriptor: bf16 x bf16 -> fp32, M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | (b_mn_major ? (1u << 16) : 0u) |
           (static_cast<uint32_t>(n >> 3) << 17) | (static_cast<uint32_t>(kTile >> 4) << 24);
}

// Optional timeline instrumentation (compiled in only with -DDDTREE_TRACE; development aid).
#ifdef DDTREE_TRACE
__device__ unsigned long long* g_trace = nullptr;
__device__ __forceinline__ void trace_mark(int idx) {
    if (g_trace) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        const int cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        g_trace[cta * 64 + idx] = t;
    }
}
#define TRACE(idx) trace_mark(idx)
__device__ __forceinline__ void trace_clk(int idx) {
    if (g_trace) {
        long long t;
        asm volatile("mov.u64 %0, %%clock64;" : "=l"(t) :: "memory");
        const int cta = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);
        g_trace[cta * 64 + idx] = static_cast<unsigned long long>(t);
    }
}
#define TRACE_CLK(idx) trace_clk(idx)
// Low-overhead time stamps: clock64 into registers for two steady-state tiles, written out once
// after the loop (a stamp that writes to global memory costs ~300 cycles and distorts the loop).
#ifndef DDTREE_STAMP_TILE
#define DDTREE_STAMP_TILE 8
#endif
constexpr int kStampTile = DDTREE_STAMP_TILE;
#define STAMP_DECL long long stamp_[16] = {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}
#define STAMP(cond, i) do { if (cond) { long long t_; asm volatile("mov.u64 %0, %%clock64;" : "=l"(t_)); stamp_[i] = t_; } } while (0)
#define STAMP_FLUSH(cond, base) do { if ((cond) && g_trace) { \
        const int cta_ = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z); \
        for (int i_ = 0; i_ < 16; ++i_) if (stamp_[i_]) g_trace[cta_ * 64 + (base) + i_] = static_cast<unsigned long long>(stamp_[i_]); } } while (0)
#else
constexpr int kStampTile = 8;
#define STAMP_DECL ((void)0)
#define STAMP(cond, i) ((void)0)
#define STAMP_FLUSH(cond, base) ((void)0)
#define TRACE(idx) ((void)0)
#define TRACE_CLK(idx) ((void)0)
#endif

struct Smem {
    uint8_t q[kTileBytes];
    uint8_t k[kStages][kTileBytes];
    uint8_t v[kStages][kTileBytes];
    uint64_t q_full, k_full[kStages], k_free[kStages], v_full[kStages], v_free[kStages];
    uint64_t s_full[kSBufs], p_ready[kSBufs][2], o_done[2], fin;
    float xm[2][kTile], xl[2][kTile]; // [column half][row]: reference maximum and sum, exchanged at the end
    uint32_t tmem_base;
    uint32_t abort;
};

struct KernelParams {
    const int32_t* cu_prefix;
    const uint32_t* anc_mask;
    const int32_t* n_rows;
    __nv_bfloat16* out;
    float* lse;
    __half* part_o;  // [S, R, Hkv, rows_pad, 128]: each split's O divided by its own sum, fp16
    float2* part_ml; // [S, R, Hkv, rows_pad] (reference max in log2 units, sum)
    uint32_t* status;
    int R, N, W, Hq, Hkv, G, splits, rows_pad;
    float scale_log2;
    // blockIdx.z -> request, longest prefix first (CTAs are dispatched in index order: the long ones must
    // not be left for the end); identity when the batch has more than kMaxOrdered requests
    int ordered;
    uint16_t order[kMaxOrdered];
};

__device__ __forceinline__ float max3(float a, float b, float c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
    return d;
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Two non-negative finite floats -> packed bf16 pair (low half = a), rounding to nearest with ties
// away from zero: add half an ulp of bf16 to the bit pattern, keep the upper 16 bits.  Done with
// integer adds and one byte permute so that it stays off the conversion/transcendental unit, which
// the exponentials already saturate.
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    return __byte_perm(__float_as_uint(a) + 0x8000u, __float_as_uint(b) + 0x8000u, 0x7632);
}

// Exponentials of score columns [kBegin, kEnd) of one thread relative to the reference m_use, packed to
// bf16 pairs (low half = even key), and their sum added to rowsum.
template <int kBegin, int kEnd>
__device__ __forceinline__ void exp_block(const uint32_t (&sv)[64], uint32_t (&pk)[32], float& rowsum, float scale_log2,
                                          float m_use) {
#pragma unroll
    for (int c = kBegin; c < kEnd; c += 2) {
        const float e0 = ex2(fmaf(__uint_as_float(sv[c]), scale_log2, -m_use));
        const float e1 = ex2(fmaf(__uint_as_float(sv[c + 1]), scale_log2, -m_use));
        rowsum += e0 + e1;
        pk[c >> 1] = pack_bf16(e0, e1);
    }
}

// Replace the scores of invisible keys by -inf: bit c of `word` tells whether key c of this
// 32-key group is visible to this row.
__device__ __forceinline__ void mask32(uint32_t (&sv)[64], int o, uint32_t word) {
#pragma unroll
    for (int c = 0; c < 32; ++c)
        if (!((word >> c) & 1u)) sv[o + c] = 0xff800000u;
}

// ---- short last row tile ----------------------------------------------------------------------
// A tree of B = 2^k nodes plus the root leaves G rows over for a last row tile of their own; run
// through the path below, that tile would cost as much as a full one (a fifth of all CTAs for B = 128,
// G = 4).  With so few rows the roles of
// rows and keys are swapped for the scores: S^T = K Q^T puts the 128 keys of a tile on the TMEM lanes
// and the (at most 16) rows on the columns, so a thread exponentiates 16 values per tile instead of
// 64, keeps its own partial row sums, and the tile costs little more than the copy of its K/V.  The
// second product is swapped as well: O^T += V^T P^T with the V tile as the 128-row (MN-major) operand
// and P^T, 16 rows x 128 keys written to shared memory by the key threads, as the narrow one; O^T
// has the head dimension on the lanes and one column per row.  A row's reference maximum is set by
// an exact reduction over the key threads on the first tile and whenever an exponential exceeds
// 2^24; otherwise the threads only meet at one barrier per tile.  Two groups of 128 key threads take
// alternate tiles, each with its own reference maxima, sums and O^T, merged at the end.  The CTA sees
// the whole KV range of its rows (the path is used only where there are no KV splits) and writes the
// output itself.  Measured: ~1200 cycles per KV tile against ~2200 on the full-tile path; the tensor
// pipe is the limit (16 instructions per tile that each stream a 4 KB operand from shared memory).
constexpr int kTailRows = 16;
constexpr int kTailKStages = 3, kTailVStages = 3;
constexpr uint32_t kTailQHalf = kTailRows * 128;  // one 64-wide half of the 16-row Q or P^T tile
constexpr int kTailSBufs = 4;    // S^T = K Q^T runs four tiles ahead of the key threads
constexpr uint32_t kColST = 0;  // S^T buffers at columns 0, 32, 64 and 96
constexpr uint32_t kColOT = 256; // O^T of key group g at column 256 + 32 g

struct TailSmem {
    uint8_t k[kTailKStages][kTileBytes];
    uint8_t v[kTailVStages][kTileBytes];
    uint8_t q[2 * kTailQHalf];      // the tile's 16 query rows
    uint8_t pt[2][2][2 * kTailQHalf];  // [group][buffer] P^T: [row][key], two 64-key halves, 128-byte swizzle (K-major operand)
    uint64_t q_full, k_full[kTailKStages], k_free[kTailKStages], v_full[kTailVStages], v_free[kTailVStages];
    // One barrier per buffer, each watched by one key group only: a parity wait must see every phase in turn.
    uint64_t s_full[kTailSBufs], p_ready[2][2], o_done[2][2];
    float red[2][4][kTailRows];  // [group][warp]: row maxima inside the loop, row sums at the end
    float mref[2][kTailRows];    // the groups' reference maxima, exchanged at the end
    uint32_t tmem_base;
    uint32_t abort;
    uint32_t key_fail[2];  // per group: a key thread's wait gave up (written before, read after a barrier of the group)
};

__device__ __forceinline__ void tail_tile_cta(const CUtensorMap* map_qt, const CUtensorMap* map_kc, const CUtensorMap* map_vc,
                                              const CUtensorMap* map_kt, const CUtensorMap* map_vt, const KernelParams& p,
                                              uint8_t* smem_raw, int kvh, int rt, int r, int n) {
    TailSmem& sm = *reinterpret_cast<TailSmem*>(smem_raw);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rows = min(n * p.G - rt * kTile, kTailRows);  // valid rows of this tile (> 0: checked by the caller)
    const int p0 = p.cu_prefix[r], P = p.cu_prefix[r + 1] - p0;
    const int prefix_tiles = (P + kTile - 1) / kTile, tree_tiles = (n + kTile - 1) / kTile;
    const int my_tiles = prefix_tiles + tree_tiles;  // the whole KV range (this path runs without KV splits), >= 1
    constexpr int t_begin = 0;

    volatile uint32_t* abort_flag = &sm.abort;
    if (tid == 0) TRACE(60);
    int k_issued = 0, v_issued = 0;
    auto tile_row = [&](int j, bool& in_prefix) {
        const int t = t_begin + j;
        in_prefix = t < prefix_tiles;
        return in_prefix ? p0 + t * kTile : r * p.N + (t - prefix_tiles) * kTile;
    };
    auto load_k = [&](int j) {
        bool in_prefix;
        const int row = tile_row(j, in_prefix), s = j % kTailKStages;
        mbar_expect_tx(smem_u32(&sm.k_full[s]), kTileBytes);
        for (int h = 0; h < 2; ++h)
            tma_load_3d(smem_u32(sm.k[s]) + h * kHalfBytes, in_prefix ? map_kc : map_kt, smem_u32(&sm.k_full[s]), h * 64, kvh, row);
    };
    auto load_v = [&](int j) {
        bool in_prefix;
        const int row = tile_row(j, in_prefix), s = j % kTailVStages;
        mbar_expect_tx(smem_u32(&sm.v_full[s]), kTileBytes);
        for (int h = 0; h < 2; ++h)
            tma_load_3d(smem_u32(sm.v[s]) + h * kHalfBytes, in_prefix ? map_vc : map_vt, smem_u32(&sm.v_full[s]), h * 64, kvh, row);
    };
    if (warp == kProducerWarp && lane == 0) {
        mbar_init(smem_u32(&sm.q_full), 1);
        for (int s = 0; s < kTailKStages; ++s) { mbar_init(smem_u32(&sm.k_full[s]), 1); mbar_init(smem_u32(&sm.k_free[s]), 1); }
        for (int s = 0; s < kTailVStages; ++s) { mbar_init(smem_u32(&sm.v_full[s]), 1); mbar_init(smem_u32(&sm.v_free[s]), 1); }
        for (int b = 0; b < kTailSBufs; ++b) mbar_init(smem_u32(&sm.s_full[b]), 1);
        for (int b = 0; b < 4; ++b) { mbar_init(smem_u32(&sm.p_ready[0][0]) + 8 * b, 1); mbar_init(smem_u32(&sm.o_done[0][0]) + 8 * b, 1); }
        sm.abort = 0;
        sm.key_fail[0] = 0;
        sm.key_fail[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const int nodes_per_tile = kTile / p.G;
        mbar_expect_tx(smem_u32(&sm.q_full), 2 * kTailQHalf);
        for (int h = 0; h < 2; ++h)
            tma_load_4d(smem_u32(sm.q) + h * kTailQHalf, map_qt, smem_u32(&sm.q_full), h * 64, 0, kvh, r * p.N + rt * nodes_per_tile);
        for (; k_issued < my_tiles && k_issued < kTailKStages; ++k_issued) load_k(k_issued);
        for (; v_issued < my_tiles && v_issued < kTailVStages; ++v_issued) load_v(v_issued);
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (tid < 256) {  // P^T starts as zeros; rows beyond the valid ones are never written
        uint4* z = reinterpret_cast<uint4*>(sm.pt);
#pragma unroll
        for (int u = 0; u < 4; ++u) z[tid + 256 * u] = make_uint4(0u, 0u, 0u, 0u);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;

    if (warp == kProducerWarp) {
        if (lane == 0) {
            // the two rings are polled independently: a copy starts as soon as its slot is free
            uint32_t idle = 0;
            while (k_issued < my_tiles || v_issued < my_tiles) {
                bool progressed = false;
                if (k_issued < my_tiles &&
                    mbar_test(smem_u32(&sm.k_free[k_issued % kTailKStages]), ((k_issued / kTailKStages) - 1) & 1)) {
                    load_k(k_issued++);
                    progressed = true;
                }
                if (v_issued < my_tiles &&
                    mbar_test(smem_u32(&sm.v_free[v_issued % kTailVStages]), ((v_issued / kTailVStages) - 1) & 1)) {
                    load_v(v_issued++);
                    progressed = true;
                }
                if (progressed) { idle = 0; continue; }
                __nanosleep(32);
                if (++idle > kSpinLimit) { *abort_flag = 1; break; }
                if ((idle & 255u) == 0 && *abort_flag) break;
            }
        }
    } else if (warp == kMmaWarp) {
        constexpr uint32_t idesc_st = instr_desc(kTailRows, false);          // 128 keys x 16 rows, both operands K-major
        constexpr uint32_t idesc_pv = instr_desc(kTailRows, false) | (1u << 15);  // 128 head-dim x 16 rows, V^T MN-major
        constexpr uint32_t kQHalf = kTailQHalf >> 4;                          // second 64-wide half of Q / P^T, descriptor units
        const uint64_t q_desc = smem_desc(smem_u32(sm.q), 16);
        const uint64_t k_desc0 = smem_desc(smem_u32(sm.k[0]), 16);
        const uint64_t v_desc0 = smem_desc(smem_u32(sm.v[0]), kHalfBytes);
        const uint64_t p_desc0 = smem_desc(smem_u32(sm.pt[0][0]), 16);
        // S^T[j % 4] = K_j Q^T: the K tile is the 128-row operand, the 16 query rows the other
        auto issue_st = [&](int j) {
            const int s = j % kTailKStages, b = j % kTailSBufs;
            const uint64_t kd = k_desc0 + static_cast<uint64_t>(s) * (kTileBytes >> 4);
            const uint32_t d_s = tmem + kColST + b * 32;
            umma_ss<false>(d_s, kd, q_desc, idesc_st);
            umma_ss<true>(d_s, kd + 2, q_desc + 2, idesc_st);
            umma_ss<true>(d_s, kd + 4, q_desc + 4, idesc_st);
            umma_ss<true>(d_s, kd + 6, q_desc + 6, idesc_st);
            umma_ss<true>(d_s, kd + 1024, q_desc + kQHalf, idesc_st);
            umma_ss<true>(d_s, kd + 1026, q_desc + kQHalf + 2, idesc_st);
            umma_ss<true>(d_s, kd + 1028, q_desc + kQHalf + 4, idesc_st);
            umma_ss<true>(d_s, kd + 1030, q_desc + kQHalf + 6, idesc_st);
            tc_commit(smem_u32(&sm.k_free[s]));
            tc_commit(smem_u32(&sm.s_full[b]));
        };
        auto wait_k = [&](int j) {
            return __all_sync(kFull, mbar_wait(smem_u32(&sm.k_full[j % kTailKStages]), (j / kTailKStages) & 1, abort_flag));
        };
        bool ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.q_full), 0, abort_flag));
        for (int j = 0; j < my_tiles && j < kTailSBufs && ok; ++j) {
            ok = wait_k(j);
            if (!ok) break;
            tc_fence_after();
            if (elect_one()) issue_st(j);
            __syncwarp();
        }
        STAMP_DECL;
        for (int j = 0; j < my_tiles && ok; ++j) {
            // One burst per tile: O_g^T += V_j^T P_j^T, then the scores of tile j+4 into the S^T buffer the key
            // threads have just read.  Every instruction streams a 128-row operand (4 KB) from shared
            // memory, which takes the tensor pipe ~50 cycles whatever the other extent, so a tile costs it
            // ~850 cycles; the barriers are tested together beforehand to keep it from draining.
            const int s = j % kTailVStages, g = j & 1, b = (j >> 1) & 1;  // key group and its P^T buffer
            const bool more = j + kTailSBufs < my_tiles;
            [[maybe_unused]] const bool st8 = j == kStampTile;
            STAMP(st8, 0);
            const bool k_ok = !more || mbar_test(smem_u32(&sm.k_full[(j + kTailSBufs) % kTailKStages]), ((j + kTailSBufs) / kTailKStages) & 1);
            const bool ready = mbar_test(smem_u32(&sm.v_full[s]), (j / kTailVStages) & 1) & k_ok &
                               mbar_test(smem_u32(&sm.p_ready[g][b]), (j >> 2) & 1);
            if (!__all_sync(kFull, ready)) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.v_full[s]), (j / kTailVStages) & 1, abort_flag)) &&
                     (!more || wait_k(j + kTailSBufs)) &&
                     __all_sync(kFull, mbar_wait(smem_u32(&sm.p_ready[g][b]), (j >> 2) & 1, abort_flag));
                if (!ok) break;
            }
            STAMP(st8, 1);
            tc_fence_after();
            const uint64_t vd = v_desc0 + static_cast<uint64_t>(s) * (kTileBytes >> 4);
            const uint64_t pd = p_desc0 + static_cast<uint64_t>(g * 2 + b) * ((2 * kTailQHalf) >> 4);
            const uint32_t d_o = tmem + kColOT + g * 32;
            if (elect_one()) {
                // 16 keys per instruction: 16 rows further in V, 32 bytes further in P^T's rows
                if (j > 1) umma_ss<true>(d_o, vd, pd, idesc_pv);
                else umma_ss<false>(d_o, vd, pd, idesc_pv);
                umma_ss<true>(d_o, vd + 128, pd + 2, idesc_pv);
                umma_ss<true>(d_o, vd + 256, pd + 4, idesc_pv);
                umma_ss<true>(d_o, vd + 384, pd + 6, idesc_pv);
                umma_ss<true>(d_o, vd + 512, pd + kQHalf, idesc_pv);
                umma_ss<true>(d_o, vd + 640, pd + kQHalf + 2, idesc_pv);
                umma_ss<true>(d_o, vd + 768, pd + kQHalf + 4, idesc_pv);
                umma_ss<true>(d_o, vd + 896, pd + kQHalf + 6, idesc_pv);
                tc_commit(smem_u32(&sm.o_done[g][b]));
                tc_commit(smem_u32(&sm.v_free[s]));
                if (more) issue_st(j + kTailSBufs);
            }
            __syncwarp();
            STAMP(st8, 2);
        }
        STAMP_FLUSH(lane == 0, 0);
    } else {
        // ---- key threads: two groups of 128 (warps 0-3: even tiles, warps 4-7: odd tiles).  Thread c of a
        //      group owns key c of its tiles and head-dim element c of the group's O^T.  A group has its own
        //      reference maxima, sums and O^T, like the column halves of the full tiles: the groups never
        //      talk inside the loop and are merged at the end like two KV splits. ----------------------
        const int g = warp >> 2, c = tid & (kTile - 1);
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const uint32_t o_addr = lane_addr + kColOT + g * 32;
        const uint32_t p_off = (c >> 6) * kTailQHalf + ((c & 7) << 1);  // + row*128 + (chunk ^ row%8)*16
        const int chunk = (c & 63) >> 3;
        const int my_count = (my_tiles - g + 1) >> 1;  // tiles g, g+2, ... of this CTA
        float mref[kTailRows], l_part[kTailRows];
#pragma unroll
        for (int i = 0; i < kTailRows; ++i) { mref[i] = -CUDART_INF_F; l_part[i] = 0.f; }
        auto store_p = [&](int b, const float (&pv)[kTailRows]) {
            uint8_t* base = sm.pt[g][b] + p_off;
#pragma unroll
            for (int i = 0; i < kTailRows; ++i)
                if (i < rows)
                    *reinterpret_cast<__nv_bfloat16*>(base + i * 128 + ((chunk ^ (i & 7)) << 4)) = __float2bfloat16_rn(pv[i]);
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        };
        // completion of the product of this group's q-th tile (it read P^T[q % 2] and added to the group's O^T)
        auto wait_pv = [&](int q) {
            return __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[g][q & 1]), (q >> 1) & 1, abort_flag));
        };
        bool failed = false;
        STAMP_DECL;
        for (int q = 0; q < my_count; ++q) {
            const int j = 2 * q + g, t = t_begin + j, b = q & 1, sb = j % kTailSBufs;
            [[maybe_unused]] const bool st8 = j == kStampTile;
            STAMP(st8, 0);
            STAMP(j == kStampTile + 2, 8);
            STAMP(j == kStampTile + 8, 9);
            STAMP(q == 0, 10);
            STAMP(q == 4, 12);
            bool ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.s_full[sb]), (j / kTailSBufs) & 1, abort_flag));
            STAMP(st8, 1);
            uint32_t sv[kTailRows];
#pragma unroll
            for (int i = 0; i < kTailRows; ++i) sv[i] = 0u;
            if (ok) {
                tc_fence_after();
                tmem_ld16(sv, lane_addr + kColST + sb * 32);
            }
            // which rows see my key
            uint32_t vis = 0;
            if (t < prefix_tiles) {
                vis = t * kTile + c < P ? 0xffffu : 0u;
            } else {
                const int kn = (t - prefix_tiles) * kTile + c;
                if (kn < n) {
#pragma unroll
                    for (int i = 0; i < kTailRows; ++i) {
                        if (i < rows) {
                            const int node = (rt * kTile + i) / p.G;
                            const uint32_t word = p.anc_mask[(static_cast<size_t>(r) * p.N + node) * p.W + (kn >> 5)];
                            vis |= ((word >> (kn & 31)) & 1u) << i;
                        }
                    }
                }
            }
            tmem_wait_ld();
            tc_fence_before();
            STAMP(st8, 2);
            float x[kTailRows], pv[kTailRows];
            bool need = false;
#pragma unroll
            for (int i = 0; i < kTailRows; ++i) {
                x[i] = ((vis >> i) & 1u) ? __uint_as_float(sv[i]) * p.scale_log2 : -CUDART_INF_F;
                pv[i] = ex2(x[i] - (mref[i] == -CUDART_INF_F ? 0.f : mref[i]));
                if (i < rows) need |= mref[i] == -CUDART_INF_F || !(pv[i] < 16777216.f);
            }
            STAMP(st8, 3);
            // P^T[b] was read by the product of this group's tile q-2
            if (ok && q > 1) ok = wait_pv(q - 2);
            STAMP(st8, 4);
            store_p(b, pv);
            STAMP(st8, 5);
            // A wait that gave up joins the vote, and the flag it left is read only after the barrier: every
            // thread of the group takes the same way out (a thread missing at a later barrier would hang the others).
            if (!ok) sm.key_fail[g] = 1;
            const bool slow = bar_keys_or(g, need || !ok);
            STAMP(st8, 6);
            if (slow) {
                if (*reinterpret_cast<volatile uint32_t*>(&sm.key_fail[g])) { failed = true; break; }
#pragma unroll
                for (int i = 0; i < kTailRows; ++i) {
                    float mx = x[i];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(kFull, mx, o));
                    if (lane == 0) sm.red[g][warp & 3][i] = mx;
                }
                bar_keys(g);
                bool bump_any = false;
                float alpha[kTailRows];
#pragma unroll
                for (int i = 0; i < kTailRows; ++i) {
                    const float m_tile = fmaxf(fmaxf(sm.red[g][0][i], sm.red[g][1][i]), fmaxf(sm.red[g][2][i], sm.red[g][3][i]));
                    const bool bump = m_tile > mref[i] + 8.f;
                    alpha[i] = bump ? ex2(mref[i] - m_tile) : 1.f;
                    if (bump) { l_part[i] *= alpha[i]; mref[i] = m_tile; }
                    if (i < rows) bump_any |= bump;
                    pv[i] = ex2(x[i] - (mref[i] == -CUDART_INF_F ? 0.f : mref[i]));
                }
                if (q > 0 && bump_any) {  // the group's O^T holds the sum over its earlier tiles: scale its columns
                    if (!wait_pv(q - 1)) sm.key_fail[g] = 1;
                    tc_fence_after();
                    uint32_t ov[kTailRows];
                    tmem_ld16(ov, o_addr);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < kTailRows; ++i) ov[i] = __float_as_uint(__uint_as_float(ov[i]) * alpha[i]);
                    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                                 ::"r"(o_addr), "r"(ov[0]), "r"(ov[1]), "r"(ov[2]), "r"(ov[3]), "r"(ov[4]), "r"(ov[5]), "r"(ov[6]),
                                   "r"(ov[7]), "r"(ov[8]), "r"(ov[9]), "r"(ov[10]), "r"(ov[11]), "r"(ov[12]), "r"(ov[13]), "r"(ov[14]), "r"(ov[15])
                                 : "memory");
                    tmem_wait_st();
                    tc_fence_before();
                }
                store_p(b, pv);
                bar_keys(g);
                if (*reinterpret_cast<volatile uint32_t*>(&sm.key_fail[g])) { failed = true; break; }
            }
#pragma unroll
            for (int i = 0; i < kTailRows; ++i) l_part[i] += pv[i];
            if (c == 0) mbar_arrive(smem_u32(&sm.p_ready[g][b]));
            STAMP(st8, 7);
        }
        STAMP(true, 11);
        STAMP_FLUSH(c == 0, g ? 32 : 16);

        // ---- epilogue: row sums over each group's threads, then group 0 merges the two groups and thread c
        //      writes head-dim element c of every row ----------------------------------------------------
        {
            bool ok = !failed;
            if (ok && my_count > 1) ok = wait_pv(my_count - 2);
            if (ok && my_count > 0) ok = wait_pv(my_count - 1);
            if (!ok) sm.key_fail[g] = 1;
#pragma unroll
            for (int i = 0; i < kTailRows; ++i) {
                float sum = l_part[i];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(kFull, sum, o);
                if (lane == 0) sm.red[g][warp & 3][i] = sum;
                if (c == i) sm.mref[g][i] = mref[i];
            }
            tc_fence_before();
            bar_all_keys();
            const volatile uint32_t* kf = sm.key_fail;
            if (g == 0 && !(kf[0] | kf[1])) {
                tc_fence_after();
                const bool two = my_tiles > 1;  // the other group had tiles: its O^T has been written
                uint32_t oa[kTailRows], ob[kTailRows];
                tmem_ld16(oa, lane_addr + kColOT);
                if (two) tmem_ld16(ob, lane_addr + kColOT + 32);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < kTailRows; ++i) {
                    if (i < rows) {
                        const float l_a = sm.red[0][0][i] + sm.red[0][1][i] + sm.red[0][2][i] + sm.red[0][3][i];
                        const float l_b = sm.red[1][0][i] + sm.red[1][1][i] + sm.red[1][2][i] + sm.red[1][3][i];
                        const float m_a = mref[i], m_b = sm.mref[1][i];
                        const float m_row = fmaxf(m_a, m_b);
                        const float w_a = m_a == -CUDART_INF_F ? 0.f : ex2(m_a - m_row);
                        const float w_b = (!two || m_b == -CUDART_INF_F) ? 0.f : ex2(m_b - m_row);
                        const float l_row = l_a * w_a + l_b * w_b;
                        const float f = l_row > 0.f ? 1.f / l_row : 0.f;
                        float o = __uint_as_float(oa[i]) * (w_a * f);
                        if (w_b > 0.f) o = fmaf(__uint_as_float(ob[i]), w_b * f, o);
                        const int grow = rt * kTile + i, node = grow / p.G;
                        const size_t head_row = (static_cast<size_t>(r) * p.N + node) * p.Hq + kvh * p.G + grow % p.G;
                        p.out[head_row * kTile + c] = __float2bfloat16_rn(o);
                        if (c == 0 && p.lse) p.lse[head_row] = (m_row + log2f(l_row)) / kLog2e;
                    }
                }
            }
        }
    }

    // ---- teardown -------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (tid == 0) TRACE(61);
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (sm.abort) {
        if (warp == kProducerWarp && lane == 0) {
            uint32_t scratch = 0;
            mbar_wait(smem_u32(&sm.q_full), 0, &scratch);
            for (int j = max(0, k_issued - kTailKStages); j < k_issued; ++j)
                mbar_wait(smem_u32(&sm.k_full[j % kTailKStages]), (j / kTailKStages) & 1, &scratch);
            for (int j = max(0, v_issued - kTailVStages); j < v_issued; ++j)
                mbar_wait(smem_u32(&sm.v_full[j % kTailVStages]), (j / kTailVStages) & 1, &scratch);
            atomicExch(p.status, kErrTimeout);
        }
        __syncthreads();
    }
}

// kShortTile: the grid's last row tile takes the short-tile path.  A kernel of its own rather than a run-time
// flag: with that path compiled in, a layer of a one-request batch (CTAs that live ~10 us) was measured
// ~2 us slower although none of its CTAs takes the path, and such batches never use it.
template <bool kShortTile>
__global__ void __launch_bounds__(kThreads, 1)
tree_attention_bf16_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                           const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kt,
                           const __grid_constant__ CUtensorMap map_vt, const __grid_constant__ CUtensorMap map_qt,
                           const KernelParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    if (smem_u32(smem_raw) & 1023u) {  // the 128-byte swizzle needs 1024-byte aligned tiles
        if (threadIdx.x == 0) atomicExch(p.status, kErrAlign);
        return;
    }

    pdl_wait();               // everything read below may come from the previous kernel of the stream
    const int split = blockIdx.x;
    const int kvh = blockIdx.y % p.Hkv, rt = blockIdx.y / p.Hkv;
    const int r = p.ordered ? p.order[blockIdx.z] : blockIdx.z;
    const int n = min(p.n_rows[r], p.N);
    if (rt * kTile >= n * p.G) return;  // whole row tile is padding
    if constexpr (kShortTile) {
        if (rt == p.rows_pad / kTile - 1) {
            tail_tile_cta(&map_qt, &map_kc, &map_vc, &map_kt, &map_vt, p, smem_raw, kvh, rt, r, n);
            return;
        }
    }
    const int p0 = p.cu_prefix[r], P = p.cu_prefix[r + 1] - p0;
    const int prefix_tiles = (P + kTile - 1) / kTile, tree_tiles = (n + kTile - 1) / kTile;
    const int tiles = prefix_tiles + tree_tiles;
    const int per = (tiles + p.splits - 1) / p.splits;
    const int t_begin = split * per, t_end = min(tiles, t_begin + per);
    const int my_tiles = max(0, t_end - t_begin);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) TRACE(0);
    const size_t part_row0 = ((static_cast<size_t>(split) * p.R + r) * p.Hkv + kvh) * p.rows_pad + rt * kTile;

    if (my_tiles == 0) {  // this split has nothing to do for this request: publish empty partials
        if (tid < kTile) p.part_ml[part_row0 + tid] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }

    // ---- set-up: the producer initialises the barriers and starts the first copies at once ----
    volatile uint32_t* abort_flag = &sm.abort;
    int k_issued = 0, v_issued = 0;  // tiles whose K / V copies were started (producer lane only)
    auto tile_row = [&](int j, bool& in_prefix) {
        const int t = t_begin + j;
        in_prefix = t < prefix_tiles;
        return in_prefix ? p0 + t * kTile : r * p.N + (t - prefix_tiles) * kTile;
    };
    auto load_k = [&](int j) {
        bool in_prefix;
        const int row = tile_row(j, in_prefix), s = j % kStages;
        mbar_expect_tx(smem_u32(&sm.k_full[s]), kTileBytes);
        for (int h = 0; h < 2; ++h)
            tma_load_3d(smem_u32(sm.k[s]) + h * kHalfBytes, in_prefix ? &map_kc : &map_kt, smem_u32(&sm.k_full[s]),
                        h * 64, kvh, row);
    };
    auto load_v = [&](int j) {
        bool in_prefix;
        const int row = tile_row(j, in_prefix), s = j % kStages;
        mbar_expect_tx(smem_u32(&sm.v_full[s]), kTileBytes);
        for (int h = 0; h < 2; ++h)
            tma_load_3d(smem_u32(sm.v[s]) + h * kHalfBytes, in_prefix ? &map_vc : &map_vt, smem_u32(&sm.v_full[s]),
                        h * 64, kvh, row);
    };
    if (warp == kProducerWarp && lane == 0) {
        mbar_init(smem_u32(&sm.q_full), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&sm.k_full[s]), 1);
            mbar_init(smem_u32(&sm.k_free[s]), 1);
            mbar_init(smem_u32(&sm.v_full[s]), 1);
            mbar_init(smem_u32(&sm.v_free[s]), 1);
        }
        for (int b = 0; b < kSBufs; ++b) {
            mbar_init(smem_u32(&sm.s_full[b]), 1);
            mbar_init(smem_u32(&sm.p_ready[b][0]), kGroupThreads);
            mbar_init(smem_u32(&sm.p_ready[b][1]), kGroupThreads);
        }
        for (int b = 0; b < 2; ++b) mbar_init(smem_u32(&sm.o_done[b]), 1);
        mbar_init(smem_u32(&sm.fin), kSoftmaxThreads);
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        const int nodes_per_tile = kTile / p.G;
        mbar_expect_tx(smem_u32(&sm.q_full), kTileBytes);
        for (int h = 0; h < 2; ++h)
            tma_load_4d(smem_u32(sm.q) + h * kHalfBytes, &map_q, smem_u32(&sm.q_full), h * 64, 0, kvh,
                        r * p.N + rt * nodes_per_tile);
        // K tiles first (the first MMAs need them), then the V tiles
        for (; k_issued < my_tiles && k_issued < kStages; ++k_issued) load_k(k_issued);
        for (; v_issued < my_tiles && v_issued < kStages; ++v_issued) load_v(v_issued);
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    if (tid == 0) TRACE(1);

    if (warp == kProducerWarp) {
        // ---- TMA producer: K ring (freed when Q K^T has read it) and V ring (freed after P V) ---
        if (lane == 0) {
            while (k_issued < my_tiles || v_issued < my_tiles) {
                if (k_issued < my_tiles) {
                    if (!mbar_wait(smem_u32(&sm.k_free[k_issued % kStages]), ((k_issued / kStages) - 1) & 1, abort_flag)) break;
                    load_k(k_issued++);
                }
                if (v_issued < my_tiles && v_issued < k_issued) {
                    if (!mbar_wait(smem_u32(&sm.v_free[v_issued % kStages]), ((v_issued / kStages) - 1) & 1, abort_flag)) break;
                    load_v(v_issued++);
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ---- MMA issuer: the whole warp walks the loop (so that addresses live in uniform
        //      registers) and one elected lane issues; Q K^T runs kSBufs tiles ahead of the softmax ----
        constexpr uint32_t idesc_qk = instr_desc(kTile, false);
        constexpr uint32_t idesc_pv = instr_desc(kTile, true);
        const uint64_t q_desc = smem_desc(smem_u32(sm.q), 16);
        const uint64_t k_desc0 = smem_desc(smem_u32(sm.k[0]), 16);
        const uint64_t v_desc0 = smem_desc(smem_u32(sm.v[0]), kHalfBytes);
        // S[j % kSBufs] = Q K_j^T: 16 head-dim elements (32 bytes) per instruction; the second 64-wide
        // half of the tiles sits 16 KB further.  Called by the elected lane only.
        auto issue_qk = [&](int j) {
            const int s = j % kStages, b = j % kSBufs;
            const uint64_t kd = k_desc0 + static_cast<uint64_t>(s) * (kTileBytes >> 4);
            const uint32_t d_s = tmem + kColS + b * kTile;
            if (j < 6) TRACE(30 + j);
            umma_ss<false>(d_s, q_desc, kd, idesc_qk);
            umma_ss<true>(d_s, q_desc + 2, kd + 2, idesc_qk);
            umma_ss<true>(d_s, q_desc + 4, kd + 4, idesc_qk);
            umma_ss<true>(d_s, q_desc + 6, kd + 6, idesc_qk);
            umma_ss<true>(d_s, q_desc + 1024, kd + 1024, idesc_qk);
            umma_ss<true>(d_s, q_desc + 1026, kd + 1026, idesc_qk);
            umma_ss<true>(d_s, q_desc + 1028, kd + 1028, idesc_qk);
            umma_ss<true>(d_s, q_desc + 1030, kd + 1030, idesc_qk);
            tc_commit(smem_u32(&sm.k_free[s]));
            tc_commit(smem_u32(&sm.s_full[b]));
        };
        auto wait_k = [&](int j) {
            return __all_sync(kFull, mbar_wait(smem_u32(&sm.k_full[j % kStages]), (j / kStages) & 1, abort_flag));
        };
        bool ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.q_full), 0, abort_flag));
        if (lane == 0) TRACE(2);
        for (int j = 0; j < my_tiles && j < kSBufs && ok; ++j) {
            ok = wait_k(j);
            if (!ok) break;
            tc_fence_after();
            if (elect_one()) issue_qk(j);
            __syncwarp();
        }
        STAMP_DECL;
        for (int j = 0; j < my_tiles && ok; ++j) {
            [[maybe_unused]] const bool st8 = j == kStampTile, st9 = j == kStampTile + 1;
            STAMP(st8 || st9, st8 ? 0 : 3);
            // One burst per tile: O_h += P_h V_h for both column halves of tile j, then the scores of
            // tile j+2 into the S buffer those P halves sat in.  The tensor pipe pays a start-up
            // latency of a few hundred cycles whenever it has drained, so bursts are kept long.
            const int s = j % kStages, b = j % kSBufs;
            const bool more = j + kSBufs < my_tiles;
            // the four tests are independent instructions: their latencies overlap, and the tensor pipe
            // drains within ~150 cycles of the last issue, so this check must be short
            const bool k_ok = !more || mbar_test(smem_u32(&sm.k_full[(j + kSBufs) % kStages]), ((j + kSBufs) / kStages) & 1);
            const bool ready = mbar_test(smem_u32(&sm.v_full[s]), (j / kStages) & 1) & k_ok &
                               mbar_test(smem_u32(&sm.p_ready[b][0]), (j / kSBufs) & 1) &
                               mbar_test(smem_u32(&sm.p_ready[b][1]), (j / kSBufs) & 1);
            if (!__all_sync(kFull, ready)) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.v_full[s]), (j / kStages) & 1, abort_flag)) &&
                     (!more || wait_k(j + kSBufs)) &&
                     __all_sync(kFull, mbar_wait(smem_u32(&sm.p_ready[b][0]), (j / kSBufs) & 1, abort_flag)) &&
                     __all_sync(kFull, mbar_wait(smem_u32(&sm.p_ready[b][1]), (j / kSBufs) & 1, abort_flag));
                if (!ok) break;
            }
            STAMP(st8 || st9, st8 ? 1 : 4);
            tc_fence_after();
            const uint64_t vd = v_desc0 + static_cast<uint64_t>(s) * (kTileBytes >> 4);
            const uint32_t a_p = tmem + kColS + b * kTile;  // bf16 P: half h in columns [64h, 64h+32)
            if (elect_one()) {
                if (j < 5) TRACE(36 + 2 * j);
                // 16 keys (16 rows of 128 bytes) per instruction; half h covers keys [64h, 64h+64) of the tile
                if (j > 0) umma_ts<true>(tmem + kColO, a_p, vd, idesc_pv);
                else umma_ts<false>(tmem + kColO, a_p, vd, idesc_pv);
                umma_ts<true>(tmem + kColO, a_p + 8, vd + 128, idesc_pv);
                umma_ts<true>(tmem + kColO, a_p + 16, vd + 256, idesc_pv);
                umma_ts<true>(tmem + kColO, a_p + 24, vd + 384, idesc_pv);
                tc_commit(smem_u32(&sm.o_done[0]));
                if (j > 0) umma_ts<true>(tmem + kColO + kTile, a_p + 64, vd + 512, idesc_pv);
                else umma_ts<false>(tmem + kColO + kTile, a_p + 64, vd + 512, idesc_pv);
                umma_ts<true>(tmem + kColO + kTile, a_p + 72, vd + 640, idesc_pv);
                umma_ts<true>(tmem + kColO + kTile, a_p + 80, vd + 768, idesc_pv);
                umma_ts<true>(tmem + kColO + kTile, a_p + 88, vd + 896, idesc_pv);
                tc_commit(smem_u32(&sm.o_done[1]));
                tc_commit(smem_u32(&sm.v_free[s]));
                if (more) issue_qk(j + kSBufs);
            }
            __syncwarp();
            STAMP(st8 || st9, st8 ? 2 : 5);
        }
        STAMP_FLUSH(lane == 0, 0);
    } else {
        // ---- softmax: 256 threads; thread (wt, half) owns key columns [64*half, 64*half+64) of row wt in
        //      every tile, with its own reference maximum, sum and O accumulator: the two halves of a
        //      row never talk until the end, where they are merged like two KV splits -----------------
        const int half = tid >> 7, wt = tid & (kTile - 1);
        const int grow = rt * kTile + wt;           // row among this KV head's rows
        const int node = grow / p.G;
        const bool valid = node < n;
        const uint32_t* mrow = p.anc_mask + (static_cast<size_t>(r) * p.N + (valid ? node : 0)) * p.W;
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
        const uint32_t o_addr = lane_addr + kColO + half * kTile;
        float m_run = -CUDART_INF_F;   // reference maximum of the exponentials, scaled log2 units
        float l_run = 0.f;
        bool ok = true;
        bool s_ready = false;    // result of the early test of s_full for the coming tile
        bool preloaded = false;  // the TMEM load of the coming tile's scores is already in flight
        uint32_t sv[64];
        STAMP_DECL;
        // ---- first tile, outside the loop: there is no reference maximum yet, so the exact maximum comes
        //      first and the exponentials are taken once (inside the loop the first tile would take the
        //      optimistic pass and then the revisit: twice the exponentials, ~0.6 us per CTA) ----------------
        {
            const uint32_t s_addr = lane_addr + kColS + half * 64;
            ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.s_full[0]), 0, abort_flag));
            if (ok) {
                tc_fence_after();
                TMEM_LD32(sv, 0, s_addr);
                TMEM_LD32(sv, 32, s_addr + 32);
                if (wt == 0) TRACE(half ? 20 : 4);
                uint32_t vis0 = kFull, vis1 = kFull;
                bool all_visible = true;
                if (t_begin < prefix_tiles) {
                    const int left = P - t_begin * kTile - half * 64;
                    if (left < 64) {
                        all_visible = false;
                        vis0 = left >= 32 ? kFull : (left <= 0 ? 0u : ((1u << left) - 1u));
                        vis1 = left >= 64 ? kFull : (left <= 32 ? 0u : ((1u << (left - 32)) - 1u));
                    }
                } else {
                    all_visible = false;
                    const int w0 = (t_begin - prefix_tiles) * 4 + half * 2;
                    vis0 = w0 < p.W ? mrow[w0] : 0u;
                    vis1 = w0 + 1 < p.W ? mrow[w0 + 1] : 0u;
                }
                tmem_wait_ld();
                if (!all_visible) { mask32(sv, 0, vis0); mask32(sv, 32, vis1); }
                float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                for (int c = 0; c < 64; c += 8)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mx4[k] = max3(mx4[k], __uint_as_float(sv[c + 2 * k]), __uint_as_float(sv[c + 2 * k + 1]));
                m_run = fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]) * p.scale_log2;  // -inf if I see no key of this tile
                const float m_use = m_run == -CUDART_INF_F ? 0.f : m_run;
                float rowsum = 0.f;
                uint32_t pk[32];
                exp_block<0, 32>(sv, pk, rowsum, p.scale_log2, m_use);
                s_ready = 1 < my_tiles && mbar_test(smem_u32(&sm.s_full[1 % kSBufs]), (1 / kSBufs) & 1);
                exp_block<32, 64>(sv, pk, rowsum, p.scale_log2, m_use);
                preloaded = __all_sync(kFull, s_ready);
                if (preloaded) {
                    tc_fence_after();
                    const uint32_t s_next = lane_addr + kColS + (1 % kSBufs) * kTile + half * 64;
                    TMEM_LD32(sv, 0, s_next);
                    TMEM_LD32(sv, 32, s_next + 32);
                }
                TMEM_ST32(s_addr, pk, 0);
                l_run = rowsum;
                tmem_wait_st();
                tc_fence_before();
                mbar_arrive(smem_u32(&sm.p_ready[0][half]));
                if (wt == 0) TRACE(half ? 21 : 6);
            }
        }
        for (int j = 1; j < my_tiles && ok; ++j) {
            const int t = t_begin + j, b = j % kSBufs;
            const uint32_t s_addr = lane_addr + kColS + b * kTile + half * 64;
            [[maybe_unused]] const bool st8 = j == kStampTile;
            STAMP(st8, 0);
            STAMP(j == kStampTile + 1, 8);
            STAMP(j == kStampTile + 2, 9);
            // Barrier tests, votes and TMEM round trips cost 150-300 cycles each, during which the two
            // softmax warps of an SM sub-partition (always in the same phase) leave it idle.  So they are
            // taken off the critical path: the barriers of the coming tile are tested in the middle of
            // this tile's exponentials, and its scores are requested from TMEM before this tile's P is
            // stored; the top of the loop normally finds the load in flight.
            if (!preloaded) {
                if (!__all_sync(kFull, s_ready)) {
                    ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.s_full[b]), (j / kSBufs) & 1, abort_flag));
                    if (!ok) break;  // warp-uniform: the TMEM loads/stores below need the whole warp
                }
                tc_fence_after();
                TMEM_LD32(sv, 0, s_addr);
                TMEM_LD32(sv, 32, s_addr + 32);
            }
            if (wt == 0 && j < 5) TRACE(half ? 20 + 2 * j : 4 + 3 * j);
            STAMP(st8, 1);
            bool saw_o_done = j == 0;  // phase j-1 of o_done must be observed exactly once per tile (see below)

            // visibility of this thread's 64 keys
            uint32_t vis0 = kFull, vis1 = kFull;
            bool all_visible = true;
            if (t < prefix_tiles) {
                const int left = P - t * kTile - half * 64;  // keys of this request in my column range
                if (left < 64) {
                    all_visible = false;
                    vis0 = left >= 32 ? kFull : (left <= 0 ? 0u : ((1u << left) - 1u));
                    vis1 = left >= 64 ? kFull : (left <= 32 ? 0u : ((1u << (left - 32)) - 1u));
                }
            } else {
                all_visible = false;
                const int w0 = (t - prefix_tiles) * 4 + half * 2;
                vis0 = w0 < p.W ? mrow[w0] : 0u;
                vis1 = w0 + 1 < p.W ? mrow[w0 + 1] : 0u;
            }
            tmem_wait_ld();
            STAMP(st8, 2);
            if (!all_visible) { mask32(sv, 0, vis0); mask32(sv, 32, vis1); }
            // Optimistic pass: exponentials relative to the reference maximum as it stands.  P keeps its
            // relative precision whatever the reference (bf16 has the exponent range of fp32), so the
            // reference only has to keep the sums away from overflow: it is revisited when a row sum
            // exceeds 2^24 (or is not finite), and on the first tile, where there is none yet.
            float rowsum = 0.f;
            uint32_t pk[32];
            {
                const float m_use = m_run == -CUDART_INF_F ? 0.f : m_run;
                exp_block<0, 32>(sv, pk, rowsum, p.scale_log2, m_use);
                // early tests of the coming tile's barriers (results are consumed further down)
                s_ready = j + 1 < my_tiles && mbar_test(smem_u32(&sm.s_full[(j + 1) % kSBufs]), ((j + 1) / kSBufs) & 1);
                if (!saw_o_done) saw_o_done = mbar_test(smem_u32(&sm.o_done[half]), (j - 1) & 1);
                exp_block<32, 64>(sv, pk, rowsum, p.scale_log2, m_use);
            }
            STAMP(st8, 3);
            const bool revisit = m_run == -CUDART_INF_F || !(rowsum < 16777216.f);
            if (__any_sync(kFull, revisit)) {
                // exact maximum of my 64 scores; the reference moves only when the maximum outgrew it by 2^8
                float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
                for (int c = 0; c < 64; c += 8)
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                        mx4[k] = max3(mx4[k], __uint_as_float(sv[c + 2 * k]), __uint_as_float(sv[c + 2 * k + 1]));
                const float m_tile = fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]) * p.scale_log2;
                const bool bump = m_tile > m_run + 8.f;
                const float alpha = bump ? ex2(m_run - m_tile) : 1.f;
                if (bump) { l_run *= alpha; m_run = m_tile; }
                if (j > 0 && __any_sync(kFull, bump)) {  // O_half holds the sum over the earlier tiles: rescale my row
                    if (!__all_sync(kFull, saw_o_done)) {
                        ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[half]), (j - 1) & 1, abort_flag));
                        if (!ok) break;
                    }
                    saw_o_done = true;
                    tc_fence_after();
#pragma unroll
                    for (int c0 = 0; c0 < 128; c0 += 32) {
                        uint32_t ov[32];
                        TMEM_LD32(ov, 0, o_addr + c0);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
                        TMEM_ST32(o_addr + c0, ov, 0);
                    }
                }
                const float m_use = m_run == -CUDART_INF_F ? 0.f : m_run;
                rowsum = 0.f;
                exp_block<0, 64>(sv, pk, rowsum, p.scale_log2, m_use);
            }
            STAMP(st8, 4);
            // the scores are consumed: request the coming tile's (other S buffer) before storing P
            preloaded = __all_sync(kFull, s_ready);
            if (preloaded) {
                tc_fence_after();
                const uint32_t s_next = lane_addr + kColS + ((j + 1) % kSBufs) * kTile + half * 64;
                TMEM_LD32(sv, 0, s_next);
                TMEM_LD32(sv, 32, s_next + 32);
            }
            TMEM_ST32(s_addr, pk, 0);
            l_run += rowsum;
            tmem_wait_st();
            STAMP(st8, 5);
            // A parity wait cannot tell phase j-1 from phase j-3: a thread that skipped phases could
            // sail through a later wait while the product it needs is still running.  So every tile
            // observes the previous tile's o_done, here at the latest (by now it has long completed).
            if (!__all_sync(kFull, saw_o_done)) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[half]), (j - 1) & 1, abort_flag));
                if (!ok) break;
            }
            STAMP(st8, 6);
            tc_fence_before();
            mbar_arrive(smem_u32(&sm.p_ready[b][half]));
            STAMP(st8, 7);
            if (wt == 0 && j < 5) TRACE(half ? 21 + 2 * j : 6 + 3 * j);
        }

        if (preloaded) tmem_wait_ld();  // only when the loop was left early: no load may outlive the TMEM allocation
        STAMP(true, 10);
        // ---- epilogue: merge the two halves and write each row's 16-bit values straight from registers ----
        for (int h = 0; h < 2 && ok; ++h)
            ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[h]), (my_tiles - 1) & 1, abort_flag));
        if (tid == 0) TRACE(46);
        STAMP(true, 11);
        const bool direct = p.splits == 1;
        if (ok) {
            tc_fence_after();
            sm.xm[half][wt] = m_run;
            sm.xl[half][wt] = l_run;
            mbar_arrive(smem_u32(&sm.fin));
            ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.fin), 0, abort_flag));
        }
        STAMP(true, 12);
        float l_row = 0.f, m_row = -CUDART_INF_F;
        if (ok) {
            const float m_o = sm.xm[half ^ 1][wt], l_o = sm.xl[half ^ 1][wt];
            m_row = fmaxf(m_run, m_o);
            const float a_self = m_run == -CUDART_INF_F ? 0.f : ex2(m_run - m_row);
            const float a_other = m_o == -CUDART_INF_F ? 0.f : ex2(m_o - m_row);
            l_row = l_run * a_self + l_o * a_other;
            const float f = l_row > 0.f ? 1.f / l_row : 0.f;  // rows leave normalised, also as split partials
            const float f0 = (half == 0 ? a_self : a_other) * f, f1 = (half == 0 ? a_other : a_self) * f;
            // this thread merges head-dim columns [64*half, 64*half+64) of its row from both accumulators,
            // rounds them to 16 bits and writes its 128 contiguous bytes itself: to the output (bf16)
            // when this CTA saw the whole KV range, else to the split partials (fp16: the rows are
            // averages of V rows, so fp16's 11 bits are finer than the bf16 rounding of the final output).
            // (An SM stores ~32 bytes per clock whatever the route: staging the rows for coalesced stores
            // or for one bulk tensor store was measured and takes the same time.)
            uint16_t* dst16;
            if (direct) {
                dst16 = reinterpret_cast<uint16_t*>(p.out) +
                        ((static_cast<size_t>(r) * p.N + (valid ? node : 0)) * p.Hq + kvh * p.G + grow % p.G) * kTile + half * 64;
            } else {
                dst16 = reinterpret_cast<uint16_t*>(p.part_o) + (part_row0 + wt) * kTile + half * 64;
            }
#pragma unroll
            for (int c0 = 0; c0 < 64; c0 += 32) {
                uint32_t o0[32], o1[32], w16[16];
                TMEM_LD32(o0, 0, lane_addr + kColO + half * 64 + c0);
                TMEM_LD32(o1, 0, lane_addr + kColO + kTile + half * 64 + c0);
                tmem_wait_ld();
                STAMP(c0 == 0, 13);
#pragma unroll
                for (int q = 0; q < 16; ++q) {
                    const float a = fmaf(__uint_as_float(o1[2 * q]), f1, __uint_as_float(o0[2 * q]) * f0);
                    const float b = fmaf(__uint_as_float(o1[2 * q + 1]), f1, __uint_as_float(o0[2 * q + 1]) * f0);
                    if (direct) {
                        const __nv_bfloat162 t2 = __floats2bfloat162_rn(a, b);
                        w16[q] = *reinterpret_cast<const uint32_t*>(&t2);
                    } else {
                        const __half2 t2 = __floats2half2_rn(a, b);
                        w16[q] = *reinterpret_cast<const uint32_t*>(&t2);
                    }
                }
                if (valid) {
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        *reinterpret_cast<uint4*>(dst16 + c0 + 8 * u) = make_uint4(w16[4 * u], w16[4 * u + 1], w16[4 * u + 2], w16[4 * u + 3]);
                }
            }
            if (half == 0 && valid) {
                if (direct) {
                    if (p.lse) p.lse[(static_cast<size_t>(r) * p.N + node) * p.Hq + kvh * p.G + grow % p.G] = (m_row + log2f(l_row)) / kLog2e;
                } else {
                    p.part_ml[part_row0 + wt] = make_float2(m_row, l_row);
                }
            }
        }
        STAMP(true, 14);
        STAMP_FLUSH(wt == 0, half ? 32 : 16);
        if (tid == 0) TRACE(47);
    }

    // ---- teardown -------------------------------------------------------------------------------
    if (tid == 0) TRACE(48);
    tc_fence_before();
    __syncthreads();
    if (tid == 0) TRACE(3);
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (sm.abort) {  // CTA-uniform after the barrier above
        if (warp == kProducerWarp && lane == 0) {
            // a wait gave up: before the CTA exits, wait (bounded) for every copy still in flight
            uint32_t scratch = 0;
            mbar_wait(smem_u32(&sm.q_full), 0, &scratch);
            for (int j = max(0, k_issued - kStages); j < k_issued; ++j)
                mbar_wait(smem_u32(&sm.k_full[j % kStages]), (j / kStages) & 1, &scratch);
            for (int j = max(0, v_issued - kStages); j < v_issued; ++j)
                mbar_wait(smem_u32(&sm.v_full[j % kStages]), (j / kStages) & 1, &scratch);
            atomicExch(p.status, kErrTimeout);
        }
        __syncthreads();
    }
}

// Merge the per-split partials of one (request, row, head): out = sum_s w_s l_s O_s / sum_s w_s l_s
// with O_s the split's normalised row and w_s = 2^(m_s - max m).  One warp per output row; lane s first fetches split s's (m, l), so
// all splits' loads are in flight together (at most 32 splits).
__global__ void __launch_bounds__(128)
combine_kernel(const KernelParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    pdl_wait();  // the split partials come from the attention kernel launched just before
    const long long task = static_cast<long long>(blockIdx.x) * 4 + warp;
    if (task >= static_cast<long long>(p.R) * p.N * p.Hq) return;
    const int h = static_cast<int>(task % p.Hq);
    const int node = static_cast<int>((task / p.Hq) % p.N);
    const int r = static_cast<int>(task / (static_cast<long long>(p.Hq) * p.N));
    const int kvh = h / p.G, grow = node * p.G + h % p.G;
    const size_t split_stride = static_cast<size_t>(p.R) * p.Hkv * p.rows_pad;
    const size_t row0 = (static_cast<size_t>(r) * p.Hkv + kvh) * p.rows_pad + grow;
    // One round trip to L2 for everything this row needs: the row count of the request, the (max, sum)
    // pairs and the rows of up to 8 splits are requested together, before any of them is looked at
    // (rows of padding nodes and of empty splits lie inside the buffer; their contents are never used).
    const __half* po = p.part_o + row0 * kTile + lane * 4;
    const int n_r = p.n_rows[r];
    float2 ml = make_float2(-CUDART_INF_F, 0.f);
    if (lane < p.splits) ml = p.part_ml[lane * split_stride + row0];
    uint2 raw[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
        raw[u] = u < p.splits ? *reinterpret_cast<const uint2*>(po + u * split_stride * kTile) : make_uint2(0u, 0u);
    if (node >= n_r) return;
    float M = ml.y > 0.f ? ml.x : -CUDART_INF_F;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
    const float w = ml.y > 0.f ? exp2f(ml.x - M) : 0.f;  // an empty split never wrote its O row
    const float wl = w * ml.y;
    float l = wl;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) l += __shfl_xor_sync(kFull, l, o);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    auto add = [&](int s, uint2 v) {
        const float ws = __shfl_sync(kFull, wl, s);
        if (ws == 0.f) return;  // warp-uniform
        const float2 o01 = __half22float2(*reinterpret_cast<const __half2*>(&v.x));
        const float2 o23 = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
        acc[0] = fmaf(ws, o01.x, acc[0]); acc[1] = fmaf(ws, o01.y, acc[1]);
        acc[2] = fmaf(ws, o23.x, acc[2]); acc[3] = fmaf(ws, o23.y, acc[3]);
    };
#pragma unroll
    for (int u = 0; u < 8; ++u)
        if (u < p.splits) add(u, raw[u]);
    for (int s = 8; s < p.splits; ++s) add(s, *reinterpret_cast<const uint2*>(po + s * split_stride * kTile));
    const float inv = 1.f / l;
    const __nv_bfloat162 b0 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv);
    const __nv_bfloat162 b1 = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
    uint2 w2;
    w2.x = *reinterpret_cast<const uint32_t*>(&b0);
    w2.y = *reinterpret_cast<const uint32_t*>(&b1);
    const size_t o = ((static_cast<size_t>(r) * p.N + node) * p.Hq + h) * kTile;
    *reinterpret_cast<uint2*>(p.out + o + lane * 4) = w2;
    if (p.lse && lane == 0) p.lse[(static_cast<size_t>(r) * p.N + node) * p.Hq + h] = (M + log2f(l)) / kLog2e;
}

// ---- host side ---------------------------------------------------------------------------------

using EncodeFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                              const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                              CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeFn encode_fn() {
    static EncodeFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeFn>(f);
    }();
    return fn;
}

struct MapKey {
    const void* base;
    uint64_t d1, d2, d3;
    uint32_t b1, b3;
    bool operator==(const MapKey& o) const {
        return base == o.base && d1 == o.d1 && d2 == o.d2 && d3 == o.d3 && b1 == o.b1 && b3 == o.b3;
    }
};
struct MapKeyHash {
    size_t operator()(const MapKey& k) const {
        size_t h = reinterpret_cast<size_t>(k.base);
        for (uint64_t v : {k.d1, k.d2, k.d3, static_cast<uint64_t>(k.b1), static_cast<uint64_t>(k.b3)})
            h = h * 0x9E3779B97F4A7C15ull + v;
        return h;
    }
};
std::mutex g_map_mutex;
std::unordered_map<MapKey, CUtensorMap, MapKeyHash> g_maps;

// bf16 tensor [rows, heads, 128] (128 contiguous) viewed as {64-wide half, heads or (g, kv), rows}.
// rank 3: box {64, 1, box_rows};  rank 4 (queries): dims {128, G, Hkv, rows}, box {64, G, 1, box_rows}.
int get_map(CUtensorMap* out, const void* base, int rank, uint64_t d1, uint64_t d2, uint64_t rows, uint32_t b1,
            uint32_t box_rows) {
    const MapKey key{base, d1, rank == 4 ? d2 : 0, rows, b1, box_rows};
    {
        std::lock_guard<std::mutex> g(g_map_mutex);
        auto it = g_maps.find(key);
        if (it != g_maps.end()) { *out = it->second; return DDTREE_OK; }
    }
    EncodeFn enc = encode_fn();
    if (!enc) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: cuTensorMapEncodeTiled is not available");
    cuuint64_t dims[4];
    cuuint64_t strides[3];
    cuuint32_t box[4], estr[4] = {1, 1, 1, 1};
    if (rank == 3) {
        dims[0] = kTile; dims[1] = d1; dims[2] = rows;
        strides[0] = kTile * 2; strides[1] = d1 * kTile * 2;
        box[0] = 64; box[1] = 1; box[2] = box_rows;
    } else {
        dims[0] = kTile; dims[1] = d1; dims[2] = d2; dims[3] = rows;
        strides[0] = kTile * 2; strides[1] = d1 * kTile * 2; strides[2] = d1 * d2 * kTile * 2;
        box[0] = 64; box[1] = b1; box[2] = 1; box[3] = box_rows;
    }
    CUtensorMap m;
    const CUresult rc = enc(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(base), dims, strides, box,
                            estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                            CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (rc != CUDA_SUCCESS) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: cuTensorMapEncodeTiled failed (%d)", (int)rc);
    {
        std::lock_guard<std::mutex> g(g_map_mutex);
        if (g_maps.size() > 4096) g_maps.clear();
        g_maps[key] = m;
    }
    *out = m;
    return DDTREE_OK;
}

struct Plan {
    int row_tiles, rows_pad, splits;
    int tail;  // the last row tile takes the short-tile path
    size_t off_ml, total;
};

Plan make_plan(const AttnArgs& a) {
    Plan pl;
    pl.row_tiles = (a.N * a.G + kTile - 1) / kTile;
    pl.rows_pad = pl.row_tiles * kTile;
    const int base = a.R * a.Hkv * pl.row_tiles;
    const int max_tiles = (a.max_prefix + kTile - 1) / kTile + (a.N + kTile - 1) / kTile;
    int s = 1;
    if (base < 148) {
        s = 148 / base;
        const int cap = (max_tiles + 1) / 2;  // at least two KV tiles per split
        if (s > cap) s = cap;
        if (s > 32) s = 32;  // the combine kernel gives one lane to each split
        if (s < 1) s = 1;
    }
    pl.splits = s;
    // The short-tile path pays off where the SMs work through several CTAs each: its KV tiles cost half
    // as much.  When all CTAs run at once (a few requests, KV splits) it does not: the data comes straight
    // from HBM, its tiles are too short to hide that latency behind three-deep rings, and it would
    // only finish after the full tiles' CTAs.
    pl.tail = (base >= 148 && a.N * a.G - (pl.row_tiles - 1) * kTile <= kTailRows && kTailRows % a.G == 0) ? 1 : 0;
    const size_t rows = static_cast<size_t>(s) * a.R * a.Hkv * pl.rows_pad;
    pl.off_ml = (rows * kTile * 2 + 255) / 256 * 256;
    pl.total = pl.off_ml + (rows * 8 + 255) / 256 * 256;
    if (s == 1) { pl.off_ml = 0; pl.total = 256; }
    return pl;
}

}  // namespace

size_t tree_attention_bf16_workspace(const AttnArgs& a, const int32_t*) { return make_plan(a).total; }

#ifdef DDTREE_TRACE
extern "C" int ddtree_debug_set_trace(void* device_buffer) {
    unsigned long long* ptr = static_cast<unsigned long long*>(device_buffer);
    return cudaMemcpyToSymbol(g_trace, &ptr, sizeof(ptr)) == cudaSuccess ? 0 : 4;
}
#endif

int launch_tree_attention_bf16(const AttnArgs& a, const int32_t* cu_prefix_host, void* ws, size_t, cudaStream_t st) {
    const Plan pl = make_plan(a);
    CUtensorMap mq, mkc, mvc, mkt, mvt, mqt;
    const uint64_t tree_rows = static_cast<uint64_t>(a.R) * a.N;
    int rc = get_map(&mq, a.q, 4, a.G, a.Hkv, tree_rows, a.G, kTile / a.G);
    if (rc) return rc;
    mqt = mq;  // the 16 query rows of a short last row tile
    if (pl.tail && (rc = get_map(&mqt, a.q, 4, a.G, a.Hkv, tree_rows, a.G, kTailRows / a.G))) return rc;
    if ((rc = get_map(&mkt, a.k_tree, 3, a.Hkv, 0, tree_rows, 1, kTile))) return rc;
    if ((rc = get_map(&mvt, a.v_tree, 3, a.Hkv, 0, tree_rows, 1, kTile))) return rc;
    if (a.total_prefix > 0) {
        if ((rc = get_map(&mkc, a.k_cache, 3, a.Hkv, 0, a.total_prefix, 1, kTile))) return rc;
        if ((rc = get_map(&mvc, a.v_cache, 3, a.Hkv, 0, a.total_prefix, 1, kTile))) return rc;
    } else {
        mkc = mkt;  // never used: no request has a prefix tile
        mvc = mvt;
    }
    KernelParams p;
    p.cu_prefix = a.cu_prefix; p.anc_mask = a.anc_mask; p.n_rows = a.n_rows;
    p.out = static_cast<__nv_bfloat16*>(a.out); p.lse = a.lse;
    p.part_o = reinterpret_cast<__half*>(ws);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(ws) + pl.off_ml);
    p.status = device_status_word();
    if (!p.status) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: no device status word");
    p.R = a.R; p.N = a.N; p.W = a.W; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.G;
    p.splits = pl.splits; p.rows_pad = pl.rows_pad;
    p.scale_log2 = a.scale * kLog2e;
    p.ordered = 0;
    if (cu_prefix_host && a.R > 1 && a.R <= kMaxOrdered) {
        std::vector<int> idx(a.R);
        for (int i = 0; i < a.R; ++i) idx[i] = i;
        std::stable_sort(idx.begin(), idx.end(), [&](int x, int y) {
            return cu_prefix_host[x + 1] - cu_prefix_host[x] > cu_prefix_host[y + 1] - cu_prefix_host[y];
        });
        for (int i = 0; i < a.R; ++i) p.order[i] = static_cast<uint16_t>(idx[i]);
        p.ordered = 1;
    }

    static const size_t smem_bytes = sizeof(Smem);
    static_assert(sizeof(TailSmem) <= sizeof(Smem), "the short-tile path lives in the same allocation");
    static_assert(sizeof(Smem) <= 232448, "exceeds the 227 KB of shared memory a CTA may opt in to");
    {   // opt in to the large dynamic shared-memory size once per device
        static std::mutex mu;
        static bool done[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> g(mu);
        if (dev < 0 || dev >= 64 || !done[dev]) {
            cudaError_t e = cudaFuncSetAttribute(tree_attention_bf16_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 static_cast<int>(smem_bytes));
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(tree_attention_bf16_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem_bytes));
            if (e != cudaSuccess)
                return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: shared memory opt-in: %s", cudaGetErrorString(e));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    dim3 grid(pl.splits, pl.row_tiles * a.Hkv, a.R);
    cudaError_t e = pl.tail
        ? launch_pdl(tree_attention_bf16_kernel<true>, grid, dim3(kThreads), smem_bytes, st, mq, mkc, mvc, mkt, mvt, mqt, p)
        : launch_pdl(tree_attention_bf16_kernel<false>, grid, dim3(kThreads), smem_bytes, st, mq, mkc, mvc, mkt, mvt, mqt, p);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: launch: %s", cudaGetErrorString(e));
    if (pl.splits > 1) {
        const long long tasks = static_cast<long long>(a.R) * a.N * a.Hq;
        e = launch_pdl(combine_kernel, dim3(static_cast<unsigned>((tasks + 3) / 4)), dim3(128), 0, st, p);
        if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: combine: %s", cudaGetErrorString(e));
    }
    return DDTREE_OK;
}

}  // namespace ddtree

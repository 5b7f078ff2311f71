// Shared pieces of the sm_100a tree-attention kernels: PTX wrappers (mbarrier, TMA, tcgen05), descriptors,
// the kernels' parameter block and the small arithmetic helpers of the softmax threads.
#pragma once
#include "common.cuh"
#include <cuda.h>
#include <cuda_fp16.h>
#include <math_constants.h>

namespace ddtree {
namespace sm100 {

constexpr int kTile = 128;            // rows per row tile, keys per KV tile, head dim
constexpr uint32_t kHalfBytes = 128 * 64 * 2;      // one 64-wide half of a 128x128 bf16 tile
constexpr uint32_t kTileBytes = 2 * kHalfBytes;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2e = 1.4426950408889634f;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kMaxOrdered = 128;
constexpr uint32_t kErrTimeout = 0x5101;
constexpr uint32_t kErrAlign = 0x5102;
constexpr int kRopeDepths = kMaxL + 1;  // a tree row sits at most kMaxL positions behind its root

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
__device__ __forceinline__ bool mbar_wait_limit(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag, uint32_t limit) {
    if (mbar_test(bar, parity)) return true;
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 32) {
            __nanosleep(64);
            if ((i & 255u) == 0 && *abort_flag) return false;
        }
    }
    *abort_flag = 1;
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
    return mbar_wait_limit(bar, parity, abort_flag, kSpinLimit);
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
// 32 contiguous bytes in one store: a full sector per request (with 16-byte stores of rows 256 bytes apart every
// request fills half a sector and an SM moves 16 instead of 32 bytes per clock).  The address must be 32-byte aligned.
__device__ __forceinline__ void st_global_256(void* p, const uint32_t (&v)[16], int o) {
    asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(v[o]), "r"(v[o + 1]), "r"(v[o + 2]),
                 "r"(v[o + 3]), "r"(v[o + 4]), "r"(v[o + 5]), "r"(v[o + 6]), "r"(v[o + 7]) : "memory");
}
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* m) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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
// Register budget of the calling warp group (all four warps of it execute this together).
template <int kRegs> __device__ __forceinline__ void regs_inc() { asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegs)); }
template <int kRegs> __device__ __forceinline__ void regs_dec() { asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegs)); }

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
// 64 consecutive columns of this thread's TMEM lane -> v[0 .. 63] (one round trip: a load in flight holds the
// warp's following instructions back, so fewer, wider loads are cheaper than several narrow ones)
__device__ __forceinline__ void tmem_ld64(uint32_t (&v)[64], uint32_t taddr) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x64.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31]), "=r"(v[32]), "=r"(v[33]), "=r"(v[34]), "=r"(v[35]), "=r"(v[36]), "=r"(v[37]), "=r"(v[38]), "=r"(v[39]), "=r"(v[40]), "=r"(v[41]), "=r"(v[42]), "=r"(v[43]), "=r"(v[44]), "=r"(v[45]), "=r"(v[46]), "=r"(v[47]), "=r"(v[48]), "=r"(v[49]), "=r"(v[50]), "=r"(v[51]), "=r"(v[52]), "=r"(v[53]), "=r"(v[54]), "=r"(v[55]), "=r"(v[56]), "=r"(v[57]), "=r"(v[58]), "=r"(v[59]), "=r"(v[60]), "=r"(v[61]), "=r"(v[62]), "=r"(v[63])
                 : "r"(taddr));
}
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

struct KernelParams {
    const int32_t* cu_prefix;
    const uint32_t* anc_mask;
    const int32_t* n_rows;
    __nv_bfloat16* out;
    float* lse;
    __half* part_o;  // [S, R, Hkv, rows_pad, 128]: each split's O divided by its own sum, fp16
    float2* part_ml; // [S, R, Hkv, rows_pad] (reference max in log2 units, sum)
    uint32_t* status;
    int R, N, W, Hq, Hkv, G, rows_pad;
    int full_tiles;   // 128-row tiles handled in pairs by the CTAs of the main path
    int pairs;        // ceil(full_tiles / 2)
    int splits;       // KV splits of a pair
    int tail;         // 1: the last 128-row tile (index full_tiles) is a short tile with a CTA of its own
    int tail_splits;  // KV splits of the short tile
    int units;        // CTAs per (request, KV head) = pairs * splits + tail * tail_splits
    int node0;        // the combine kernel covers nodes node0 .. N-1
    float scale_log2;
    // rotary encoding applied on the way into the products (ddtree_tree_attention_rope): position ids of the tree rows
    // and, per request and depth, cos / sin of position x frequency for the 64 frequency pairs of a head
    const int32_t* position_ids;  // [R, N]
    const float2* rope_table;     // [R, kRopeDepths, 64] (cos, sin), depth = position - position of the request's root
    // grid index -> request, longest prefix first (CTAs are dispatched in index order: the long ones must
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

// Two non-negative floats -> packed bf16 pair (low half = a), round to nearest even.
__device__ __forceinline__ uint32_t pack_cvt(float a, float b) {
    uint32_t r;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(b), "f"(a));
    return r;
}

// Exponentials of the 64 scores of half a tile relative to the reference m_use, packed to bf16 pairs
// (pk[c] = keys 2c, 2c+1 of the half, c < 32); returns their sum.
__device__ __forceinline__ float exp_pack_64(const uint32_t (&x)[64], uint32_t (&pk)[32], float scale_log2, float m_use) {
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll
    for (int c = 0; c < 64; c += 4) {
        const float e0 = ex2(fmaf(__uint_as_float(x[c]), scale_log2, -m_use));
        const float e1 = ex2(fmaf(__uint_as_float(x[c + 1]), scale_log2, -m_use));
        const float e2 = ex2(fmaf(__uint_as_float(x[c + 2]), scale_log2, -m_use));
        const float e3 = ex2(fmaf(__uint_as_float(x[c + 3]), scale_log2, -m_use));
        s0 += e0; s1 += e1; s2 += e2; s3 += e3;
        pk[c >> 1] = pack_cvt(e0, e1);
        pk[(c >> 1) + 1] = pack_cvt(e2, e3);
    }
    return (s0 + s1) + (s2 + s3);
}

__device__ __forceinline__ float max_64(const uint32_t (&x)[64]) {
    float mx4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int c = 0; c < 64; c += 8)
#pragma unroll
        for (int k = 0; k < 4; ++k)
            mx4[k] = max3(mx4[k], __uint_as_float(x[c + 2 * k]), __uint_as_float(x[c + 2 * k + 1]));
    return fmaxf(max3(mx4[0], mx4[1], mx4[2]), mx4[3]);
}

// Replace the scores of invisible keys by -inf: bit c of `word` tells whether key o + c is visible to this row.
template <int kN>
__device__ __forceinline__ void mask32(uint32_t (&sv)[kN], int o, uint32_t word) {
#pragma unroll
    for (int c = 0; c < 32; ++c)
        if (!((word >> c) & 1u)) sv[o + c] = 0xff800000u;
}

// Number of keys of KV tile t (absolute index within the request) that any row may see: the rows of a
// staged V tile from there on belong to another request, to padding or to nobody.
__device__ __forceinline__ int keys_in_tile(int t, int prefix_tiles, int P, int n) {
    return t < prefix_tiles ? min(kTile, P - t * kTile) : min(kTile, n - (t - prefix_tiles) * kTile);
}
// Zero rows [first, 128) of a staged V tile (both 64-wide halves; the 128-byte swizzle permutes 16-byte
// chunks inside a row only).  Whole warp; the writes are made visible to the tensor pipe.
__device__ __forceinline__ void clear_v_rows(uint8_t* tile, int first, int lane) {
    const int chunks = (kTile - first) * 16;
    for (int i = lane; i < chunks; i += 32) {
        const int row = first + (i >> 4), c = i & 15;
        *reinterpret_cast<uint4*>(tile + (c >> 3) * kHalfBytes + row * 128 + (c & 7) * 16) = make_uint4(0u, 0u, 0u, 0u);
    }
    fence_async_smem();
    __syncwarp();
}
}  // namespace sm100

// The kernel for batches that leave SMs idle unless the KV range is split finely: one CTA per (request, KV head,
// 128-row tile, KV split), two threads per row (tree_attention_sm100_halves.cu).  Grid = (splits, Hkv x row tiles, R).
cudaError_t tree_attention_halves_opt_in();
cudaError_t launch_tree_attention_halves(dim3 grid, const CUtensorMap& map_q, const CUtensorMap& map_kc, const CUtensorMap& map_vc,
                                         const CUtensorMap& map_kt, const CUtensorMap& map_vt, const sm100::KernelParams& p,
                                         cudaStream_t st);
}  // namespace ddtree

// bf16 tree attention for sm_100a: split-KV flash-decoding with TMA-staged K/V tiles and tcgen05
// MMAs accumulating in tensor memory (Section 4.4: every tree row attends to the cached prefix
// and, inside the tree, to the rows named by its ancestor mask).
//
// Rows of one KV head are the (node, g) pairs of its G = Hq/Hkv query heads, row = node*G + g, so
// that budget x G rows share each K/V tile and QK^T / PV are dense 128x128x128 contractions.
//
// One CTA = one (request, KV head, 128-row tile, KV split).  Warp roles:
//   warps 0-3  softmax: thread t owns row t (= TMEM lane t): scale, mask, online max/sum, P -> TMEM
//   warp 4     TMA producer: Q once, then K/V tiles through a 3-stage ring
//   warp 5     MMA issuer: S = Q K^T (operands in shared memory), O += P V (P read from TMEM,
//              V as an MN-major shared-memory operand); owns the TMEM allocation
// The ancestor bitmask is applied only on tree tiles; prefix tiles need at most a length test on
// the request's last tile.  Each split writes un-normalised fp32 partials; a combine kernel merges
// them by log-sum-exp.  Every wait is bounded: when one gives up, the CTA raises a flag in the
// device status word, drains its copies and leaves without touching its outputs.
#include "common.cuh"
#include <cuda.h>
#include <math_constants.h>
#include <mutex>
#include <unordered_map>
#include <vector>

namespace ddtree {
namespace {

constexpr int kTile = 128;            // rows per CTA, keys per KV tile, head dim
constexpr int kStages = 3;
constexpr int kSoftmaxThreads = 128;
constexpr int kThreads = 192;
constexpr uint32_t kHalfBytes = 128 * 64 * 2;      // one 64-wide half of a 128x128 bf16 tile
constexpr uint32_t kTileBytes = 2 * kHalfBytes;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;         // S buffers at columns 0 and 128 (P aliases the first 64 of each)
constexpr uint32_t kColO = 256;
constexpr uint32_t kSpinLimit = 1u << 22;
constexpr float kLog2e = 1.4426950408889634f;
constexpr unsigned kFull = 0xffffffffu;
constexpr uint32_t kErrTimeout = 0x5101;

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
// Bounded wait.  Returns false when it gave up (or another thread of the CTA already did).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag) {
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
__device__ __forceinline__ void prefetch_tensormap(const CUtensorMap* map) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(map) : "memory");
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] * B[smem desc]
__device__ __forceinline__ void umma_ss(uint32_t d, uint64_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d), "l"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc]
__device__ __forceinline__ void umma_ts(uint32_t d, uint32_t a, uint64_t b, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(d), "r"(a), "l"(b), "r"(idesc), "r"(accumulate) : "memory");
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

struct Smem {
    uint8_t q[kTileBytes];
    uint8_t k[kStages][kTileBytes];
    uint8_t v[kStages][kTileBytes];
    uint64_t q_full, k_full[kStages], v_full[kStages], kv_free[kStages], s_full[2], p_ready[2], o_done;
    uint32_t tmem_base;
    uint32_t abort;
};

struct KernelParams {
    const int32_t* cu_prefix;
    const uint32_t* anc_mask;
    const int32_t* n_rows;
    __nv_bfloat16* out;
    float* lse;
    float* part_o;   // [S, R, Hkv, rows_pad, 128]
    float2* part_ml; // [S, R, Hkv, rows_pad] (scaled max in log2 units, sum)
    uint32_t* status;
    int R, N, W, Hq, Hkv, G, splits, rows_pad;
    float scale_log2;
};

__global__ void __launch_bounds__(kThreads, 1)
tree_attention_bf16_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                           const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kt,
                           const __grid_constant__ CUtensorMap map_vt, const KernelParams p) {
    extern __shared__ uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));

    const int split = blockIdx.x;
    const int kvh = blockIdx.y % p.Hkv, rt = blockIdx.y / p.Hkv;
    const int r = blockIdx.z;
    const int n = min(p.n_rows[r], p.N);
    if (rt * kTile >= n * p.G) return;  // whole row tile is padding
    const int p0 = p.cu_prefix[r], P = p.cu_prefix[r + 1] - p0;
    const int prefix_tiles = (P + kTile - 1) / kTile, tree_tiles = (n + kTile - 1) / kTile;
    const int tiles = prefix_tiles + tree_tiles;
    const int per = (tiles + p.splits - 1) / p.splits;
    const int t_begin = split * per, t_end = min(tiles, t_begin + per);
    const int my_tiles = max(0, t_end - t_begin);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t part_row0 = ((static_cast<size_t>(split) * p.R + r) * p.Hkv + kvh) * p.rows_pad + rt * kTile;

    if (my_tiles == 0) {  // this split has nothing to do for this request: publish empty partials
        if (tid < kTile) p.part_ml[part_row0 + tid] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }

    // ---- set-up -------------------------------------------------------------------------------
    if (tid == 0) {
        mbar_init(smem_u32(&sm.q_full), 1);
        for (int s = 0; s < kStages; ++s) {
            mbar_init(smem_u32(&sm.k_full[s]), 1);
            mbar_init(smem_u32(&sm.v_full[s]), 1);
            mbar_init(smem_u32(&sm.kv_free[s]), 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&sm.s_full[b]), 1);
            mbar_init(smem_u32(&sm.p_ready[b]), kSoftmaxThreads);
        }
        mbar_init(smem_u32(&sm.o_done), 1);
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 5) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sm.tmem_base;
    volatile uint32_t* abort_flag = &sm.abort;
    int issued = 0;  // K/V tiles whose copies were started (producer lane only)

    if (warp == 4) {
        // ---- TMA producer ---------------------------------------------------------------------
        if (lane == 0) {
            prefetch_tensormap(&map_q);
            prefetch_tensormap(prefix_tiles ? &map_kc : &map_kt);
            const int nodes_per_tile = kTile / p.G;
            mbar_expect_tx(smem_u32(&sm.q_full), kTileBytes);
            for (int h = 0; h < 2; ++h)
                tma_load_4d(smem_u32(sm.q) + h * kHalfBytes, &map_q, smem_u32(&sm.q_full), h * 64, 0, kvh,
                            r * p.N + rt * nodes_per_tile);
            bool ok = true;
            for (int j = 0; j < my_tiles && ok; ++j) {
                const int s = j % kStages, t = t_begin + j;
                if (j >= kStages) ok = mbar_wait(smem_u32(&sm.kv_free[s]), ((j / kStages) - 1) & 1, abort_flag);
                if (!ok) break;
                const bool in_prefix = t < prefix_tiles;
                const CUtensorMap* mk = in_prefix ? &map_kc : &map_kt;
                const CUtensorMap* mv = in_prefix ? &map_vc : &map_vt;
                const int row = in_prefix ? p0 + t * kTile : r * p.N + (t - prefix_tiles) * kTile;
                mbar_expect_tx(smem_u32(&sm.k_full[s]), kTileBytes);
                for (int h = 0; h < 2; ++h)
                    tma_load_3d(smem_u32(sm.k[s]) + h * kHalfBytes, mk, smem_u32(&sm.k_full[s]), h * 64, kvh, row);
                mbar_expect_tx(smem_u32(&sm.v_full[s]), kTileBytes);
                for (int h = 0; h < 2; ++h)
                    tma_load_3d(smem_u32(sm.v[s]) + h * kHalfBytes, mv, smem_u32(&sm.v_full[s]), h * 64, kvh, row);
                issued = j + 1;
            }
        }
    } else if (warp == 5) {
        // ---- MMA issuer -----------------------------------------------------------------------
        if (lane == 0) {
            constexpr uint32_t idesc_qk = instr_desc(kTile, false);
            constexpr uint32_t idesc_pv = instr_desc(kTile, true);
            bool ok = mbar_wait(smem_u32(&sm.q_full), 0, abort_flag);
            const uint32_t q_addr = smem_u32(sm.q);
            for (int j = 0; j <= my_tiles && ok; ++j) {
                if (j < my_tiles) {  // S[j&1] = Q K_j^T
                    const int s = j % kStages;
                    ok = mbar_wait(smem_u32(&sm.k_full[s]), (j / kStages) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t k_addr = smem_u32(sm.k[s]);
                    const uint32_t d_s = tmem + kColS + (j & 1) * kTile;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk) {
                        const uint32_t off = (kk >> 2) * kHalfBytes + (kk & 3) * 32;
                        umma_ss(d_s, smem_desc(q_addr + off, 16), smem_desc(k_addr + off, 16), idesc_qk, kk > 0);
                    }
                    tc_commit(smem_u32(&sm.s_full[j & 1]));
                }
                if (j > 0) {  // O += P_{j-1} V_{j-1}
                    const int i = j - 1, s = i % kStages;
                    ok = mbar_wait(smem_u32(&sm.p_ready[i & 1]), (i >> 1) & 1, abort_flag) &&
                         mbar_wait(smem_u32(&sm.v_full[s]), (i / kStages) & 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t v_addr = smem_u32(sm.v[s]);
                    const uint32_t a_p = tmem + kColS + (i & 1) * kTile;
#pragma unroll
                    for (int kk = 0; kk < 8; ++kk)  // 16 keys per instruction
                        umma_ts(tmem + kColO, a_p + kk * 8, smem_desc(v_addr + kk * 2048, kHalfBytes), idesc_pv,
                                (i > 0 || kk > 0));
                    tc_commit(smem_u32(&sm.kv_free[s]));
                    tc_commit(smem_u32(&sm.o_done));
                }
            }
        }
    } else {
        // ---- softmax warps: thread `tid` owns row `tid` of the tile ---------------------------
        const int grow = rt * kTile + tid;          // row among this KV head's rows
        const int node = grow / p.G, g = grow % p.G;
        const bool valid = node < n;
        const uint32_t* mrow = p.anc_mask + (static_cast<size_t>(r) * p.N + (valid ? node : 0)) * p.W;
        const uint32_t lane_addr = tmem + (static_cast<uint32_t>(warp * 32) << 16);
        float m_run = -CUDART_INF_F;   // running maximum, in scaled log2 units
        float l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < my_tiles && ok; ++j) {
            const int t = t_begin + j;
            const uint32_t s_addr = lane_addr + kColS + (j & 1) * kTile;
            ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.s_full[j & 1]), (j >> 1) & 1, abort_flag));
            if (!ok) break;  // warp-uniform: the TMEM loads/stores below need the whole warp
            tc_fence_after();
            uint32_t sv[128];
            TMEM_LD32(sv, 0, s_addr);
            TMEM_LD32(sv, 32, s_addr + 32);
            TMEM_LD32(sv, 64, s_addr + 64);
            TMEM_LD32(sv, 96, s_addr + 96);
            tmem_wait_ld();

            // visibility of the 128 keys of this tile for this row
            uint32_t vis[4] = {kFull, kFull, kFull, kFull};
            bool all_visible = true;
            if (t < prefix_tiles) {
                const int left = P - t * kTile;  // keys of this request in the tile
                if (left < kTile) {
                    all_visible = false;
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const int c = left - w * 32;
                        vis[w] = c >= 32 ? kFull : (c <= 0 ? 0u : ((1u << c) - 1u));
                    }
                }
            } else {
                all_visible = false;
                const int w0 = (t - prefix_tiles) * 4;
#pragma unroll
                for (int w = 0; w < 4; ++w) vis[w] = (w0 + w < p.W) ? mrow[w0 + w] : 0u;
            }
            float mx = -CUDART_INF_F;
            if (all_visible) {
#pragma unroll
                for (int c = 0; c < 128; ++c) mx = fmaxf(mx, __uint_as_float(sv[c]));
            } else {
#pragma unroll
                for (int c = 0; c < 128; ++c) {
                    const float x = ((vis[c >> 5] >> (c & 31)) & 1u) ? __uint_as_float(sv[c]) : -CUDART_INF_F;
                    sv[c] = __float_as_uint(x);
                    mx = fmaxf(mx, x);
                }
            }
            const float m_new = fmaxf(m_run, mx * p.scale_log2);
            const float m_use = m_new == -CUDART_INF_F ? 0.f : m_new;
            float rowsum = 0.f;
            uint32_t pk[64];
#pragma unroll
            for (int c = 0; c < 128; c += 2) {
                const float e0 = exp2f(fmaf(__uint_as_float(sv[c]), p.scale_log2, -m_use));
                const float e1 = exp2f(fmaf(__uint_as_float(sv[c + 1]), p.scale_log2, -m_use));
                rowsum += e0 + e1;
                const __nv_bfloat162 b = __floats2bfloat162_rn(e0, e1);  // low half = even key
                pk[c >> 1] = *reinterpret_cast<const uint32_t*>(&b);
            }
            TMEM_ST32(s_addr, pk, 0);
            TMEM_ST32(s_addr + 32, pk, 32);

            const float alpha = m_run == -CUDART_INF_F ? 1.f : exp2f(m_run - m_new);
            l_run = l_run * alpha + rowsum;
            m_run = m_new;
            if (j > 0) {
                // O holds the sum up to tile j-1: wait for that product, then rescale if the maximum moved
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done), (j - 1) & 1, abort_flag));
                if (!ok) break;
                tc_fence_after();
                if (__any_sync(kFull, alpha != 1.f)) {
#pragma unroll
                    for (int c0 = 0; c0 < 128; c0 += 32) {
                        uint32_t ov[32];
                        TMEM_LD32(ov, 0, lane_addr + kColO + c0);
                        tmem_wait_ld();
#pragma unroll
                        for (int c = 0; c < 32; ++c) ov[c] = __float_as_uint(__uint_as_float(ov[c]) * alpha);
                        TMEM_ST32(lane_addr + kColO + c0, ov, 0);
                    }
                }
            }
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&sm.p_ready[j & 1]));
        }
        // ---- epilogue ---------------------------------------------------------------------------
        if (ok) ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done), (my_tiles - 1) & 1, abort_flag));
        if (ok) {
            tc_fence_after();
            const bool direct = p.splits == 1;
            const float inv = l_run > 0.f ? 1.f / l_run : 0.f;
            const size_t orow = ((static_cast<size_t>(r) * p.N + node) * p.Hq + kvh * p.G + g) * kTile;
#pragma unroll
            for (int c0 = 0; c0 < 128; c0 += 32) {
                uint32_t ov[32];
                TMEM_LD32(ov, 0, lane_addr + kColO + c0);
                tmem_wait_ld();
                if (direct) {
                    if (valid) {
                        uint4* dst = reinterpret_cast<uint4*>(p.out + orow + c0);
#pragma unroll
                        for (int v4 = 0; v4 < 4; ++v4) {
                            uint32_t w[4];
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const __nv_bfloat162 b = __floats2bfloat162_rn(
                                    __uint_as_float(ov[v4 * 8 + 2 * e]) * inv, __uint_as_float(ov[v4 * 8 + 2 * e + 1]) * inv);
                                w[e] = *reinterpret_cast<const uint32_t*>(&b);
                            }
                            dst[v4] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                    }
                } else if (valid) {
                    float4* dst = reinterpret_cast<float4*>(p.part_o + (part_row0 + tid) * kTile + c0);
#pragma unroll
                    for (int v4 = 0; v4 < 8; ++v4)
                        dst[v4] = make_float4(__uint_as_float(ov[v4 * 4]), __uint_as_float(ov[v4 * 4 + 1]),
                                              __uint_as_float(ov[v4 * 4 + 2]), __uint_as_float(ov[v4 * 4 + 3]));
                }
            }
            if (direct) {
                if (valid && p.lse)
                    p.lse[(static_cast<size_t>(r) * p.N + node) * p.Hq + kvh * p.G + g] = (m_run + log2f(l_run)) / kLog2e;
            } else {
                p.part_ml[part_row0 + tid] = make_float2(m_run, l_run);
            }
        }
    }

    // ---- teardown -------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
    if (warp == 5) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
    if (sm.abort) {  // CTA-uniform after the barrier above
        if (warp == 4 && lane == 0) {
            // a wait gave up: before the CTA exits, wait (bounded) for every copy still in flight
            uint32_t scratch = 0;
            mbar_wait(smem_u32(&sm.q_full), 0, &scratch);
            for (int j = max(0, issued - kStages); j < issued; ++j) {
                mbar_wait(smem_u32(&sm.k_full[j % kStages]), (j / kStages) & 1, &scratch);
                mbar_wait(smem_u32(&sm.v_full[j % kStages]), (j / kStages) & 1, &scratch);
            }
            atomicExch(p.status, kErrTimeout);
        }
        __syncthreads();
    }
}

// Merge the per-split partials of one (request, row, head): out = sum_s w_s O_s / sum_s w_s l_s
// with w_s = 2^(m_s - max m).
__global__ void __launch_bounds__(128)
combine_kernel(const KernelParams p) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const long long task = static_cast<long long>(blockIdx.x) * 4 + warp;
    if (task >= static_cast<long long>(p.R) * p.N * p.Hq) return;
    const int h = static_cast<int>(task % p.Hq);
    const int node = static_cast<int>((task / p.Hq) % p.N);
    const int r = static_cast<int>(task / (static_cast<long long>(p.Hq) * p.N));
    if (node >= p.n_rows[r]) return;
    const int kvh = h / p.G, grow = node * p.G + h % p.G;
    float M = -CUDART_INF_F;
    for (int s = 0; s < p.splits; ++s)
        M = fmaxf(M, p.part_ml[((static_cast<size_t>(s) * p.R + r) * p.Hkv + kvh) * p.rows_pad + grow].x);
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    float l = 0.f;
    for (int s = 0; s < p.splits; ++s) {
        const size_t row = ((static_cast<size_t>(s) * p.R + r) * p.Hkv + kvh) * p.rows_pad + grow;
        const float2 ml = p.part_ml[row];
        if (ml.y == 0.f) continue;  // empty split: its O row was never written
        const float w = exp2f(ml.x - M);
        l += w * ml.y;
        const float4 o = *reinterpret_cast<const float4*>(p.part_o + row * kTile + lane * 4);
        acc[0] += w * o.x; acc[1] += w * o.y; acc[2] += w * o.z; acc[3] += w * o.w;
    }
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
        if (s < 1) s = 1;
    }
    pl.splits = s;
    const size_t rows = static_cast<size_t>(s) * a.R * a.Hkv * pl.rows_pad;
    pl.off_ml = (rows * kTile * 4 + 255) / 256 * 256;
    pl.total = pl.off_ml + (rows * 8 + 255) / 256 * 256;
    if (s == 1) { pl.off_ml = 0; pl.total = 256; }
    return pl;
}

}  // namespace

size_t tree_attention_bf16_workspace(const AttnArgs& a, const int32_t*) { return make_plan(a).total; }

int launch_tree_attention_bf16(const AttnArgs& a, const int32_t*, void* ws, size_t, cudaStream_t st) {
    const Plan pl = make_plan(a);
    CUtensorMap mq, mkc, mvc, mkt, mvt;
    const uint64_t tree_rows = static_cast<uint64_t>(a.R) * a.N;
    int rc = get_map(&mq, a.q, 4, a.G, a.Hkv, tree_rows, a.G, kTile / a.G);
    if (rc) return rc;
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
    p.part_o = reinterpret_cast<float*>(ws);
    p.part_ml = reinterpret_cast<float2*>(static_cast<char*>(ws) + pl.off_ml);
    p.status = device_status_word();
    if (!p.status) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: no device status word");
    p.R = a.R; p.N = a.N; p.W = a.W; p.Hq = a.Hq; p.Hkv = a.Hkv; p.G = a.G;
    p.splits = pl.splits; p.rows_pad = pl.rows_pad;
    p.scale_log2 = a.scale * kLog2e;

    static const size_t smem_bytes = sizeof(Smem) + 1024;
    {   // opt in to the large dynamic shared-memory size once per device
        static std::mutex mu;
        static bool done[64] = {};
        int dev = 0;
        cudaGetDevice(&dev);
        std::lock_guard<std::mutex> g(mu);
        if (dev < 0 || dev >= 64 || !done[dev]) {
            const cudaError_t e = cudaFuncSetAttribute(tree_attention_bf16_kernel,
                                                       cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                       static_cast<int>(smem_bytes));
            if (e != cudaSuccess)
                return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: shared memory opt-in: %s", cudaGetErrorString(e));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    dim3 grid(pl.splits, pl.row_tiles * a.Hkv, a.R);
    tree_attention_bf16_kernel<<<grid, kThreads, smem_bytes, st>>>(mq, mkc, mvc, mkt, mvt, p);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: launch: %s", cudaGetErrorString(e));
    if (pl.splits > 1) {
        const long long tasks = static_cast<long long>(a.R) * a.N * a.Hq;
        combine_kernel<<<static_cast<unsigned>((tasks + 3) / 4), 128, 0, st>>>(p);
        e = cudaGetLastError();
        if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: combine: %s", cudaGetErrorString(e));
    }
    return DDTREE_OK;
}

}  // namespace ddtree

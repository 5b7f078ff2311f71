// bf16 tree attention for sm_100a, the kernel for batches whose row tiles do not fill the SMs: one CTA =
// one (request, KV head, 128-row tile, KV split), so that a fine split of the KV range costs one 128-row
// partial per CTA (Section 4.4: every tree row attends to the cached prefix and, inside the tree, to the
// rows named by its ancestor mask).  Rows, tiles, masks and split partials are those of
// tree_attention_sm100.cu, whose combine kernel merges the splits.  Warp roles:
//   warps 0-7  softmax: two threads per row, each owns 64 key columns of every KV tile with its own reference
//              maximum, sum and O accumulator in tensor memory (no exchange per tile; merged at the end)
//   warp 8     TMA producer: Q once, then separate three-deep rings of K and V tiles
//   warp 9     MMA issuer; owns the TMEM allocation.  One burst per KV tile: O_h += P_h V_j for both column
//              halves, then the scores of tile j+2 into the score buffer those P halves sat in
//   warp 10    clears the rows of a staged V tile that belong to no visible key
// Tensor memory: two score buffers (128 columns each; a half's bf16 probabilities overwrite the first 32
// columns of its own scores), the two halves' O accumulators (128 columns each).
// With few KV tiles per CTA the fixed costs decide (set-up, the first tile, the epilogue, the partial rows
// written and merged): per KV tile and row tile this kernel costs what the two-row-tile kernel costs, but
// a CTA of that kernel writes twice the partial rows for the same number of resident CTAs.
#include "sm100_attention.cuh"

namespace ddtree {
namespace {
using namespace sm100;

constexpr int kStages = 3;
constexpr int kSBufs = 2;              // score buffers in TMEM: Q K^T runs one tile ahead of the softmax
constexpr int kSoftmaxThreads = 256;   // two threads per row, 64 key columns each
constexpr int kGroupThreads = 128;     // threads of one column half
constexpr int kProducerWarp = 8, kMmaWarp = 9, kFixWarp = 10;
constexpr int kThreads = 352;
constexpr uint32_t kColS = 0;         // S buffers at columns 0 and 128; half h's bf16 P overwrites columns [64h, 64h+32)
constexpr uint32_t kColO = 256;       // O accumulators of the two column halves at columns 256 and 384

struct Smem {
    uint8_t q[kTileBytes];
    uint8_t k[kStages][kTileBytes];
    uint8_t v[kStages][kTileBytes];
    uint64_t q_full, k_full[kStages], k_free[kStages], v_full[kStages], v_free[kStages], v_fix[kStages];
    uint64_t s_full[kSBufs], p_ready[kSBufs][2], o_done[2], fin;
    float xm[2][kTile], xl[2][kTile]; // [column half][row]: reference maximum and sum, exchanged at the end
    uint32_t tmem_base;
    uint32_t abort;
};

// Two non-negative finite floats -> packed bf16 pair (low half = a), rounding to nearest with ties
// away from zero: add half an ulp of bf16 to the bit pattern, keep the upper 16 bits.  Integer adds and
// one byte permute: it stays off the conversion/transcendental unit, which the exponentials saturate.
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

__global__ void __launch_bounds__(kThreads, 1)
tree_attention_halves_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                           const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kt,
                           const __grid_constant__ CUtensorMap map_vt, const __grid_constant__ KernelParams p) {
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
            mbar_init(smem_u32(&sm.v_fix[s]), 1);
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
    } else if (warp == kFixWarp) {
        // ---- V clean-up: every staged V tile passes through this warp on its way to the MMA warp; rows that
        //      no row may see (the ragged end of a prefix, tree rows past n_rows) are cleared: their
        //      probabilities are zero, but 0 x NaN is not.  The copies run tiles ahead of the products. ----
        for (int j = 0; j < my_tiles; ++j) {
            const int s = j % kStages;
            if (!__all_sync(kFull, mbar_wait(smem_u32(&sm.v_full[s]), (j / kStages) & 1, abort_flag))) break;
            const int first = keys_in_tile(t_begin + j, prefix_tiles, P, n);
            if (first < kTile) clear_v_rows(sm.v[s], first, lane);
            if (lane == 0) mbar_arrive(smem_u32(&sm.v_fix[s]));
            __syncwarp();
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
        for (int j = 0; j < my_tiles && j < kSBufs && ok; ++j) {
            ok = wait_k(j);
            if (!ok) break;
            tc_fence_after();
            if (elect_one()) issue_qk(j);
            __syncwarp();
        }
        for (int j = 0; j < my_tiles && ok; ++j) {
            // One burst per tile: O_h += P_h V_h for both column halves of tile j, then the scores of
            // tile j+2 into the S buffer those P halves sat in.  The tensor pipe pays a start-up
            // latency of a few hundred cycles whenever it has drained, so bursts are kept long.
            const int s = j % kStages, b = j % kSBufs;
            const bool more = j + kSBufs < my_tiles;
            // the four tests are independent instructions: their latencies overlap, and the tensor pipe
            // drains within ~150 cycles of the last issue, so this check must be short
            const bool k_ok = !more || mbar_test(smem_u32(&sm.k_full[(j + kSBufs) % kStages]), ((j + kSBufs) / kStages) & 1);
            const bool ready = mbar_test(smem_u32(&sm.v_fix[s]), (j / kStages) & 1) & k_ok &
                               mbar_test(smem_u32(&sm.p_ready[b][0]), (j / kSBufs) & 1) &
                               mbar_test(smem_u32(&sm.p_ready[b][1]), (j / kSBufs) & 1);
            if (!__all_sync(kFull, ready)) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.v_fix[s]), (j / kStages) & 1, abort_flag)) &&
                     (!more || wait_k(j + kSBufs)) &&
                     __all_sync(kFull, mbar_wait(smem_u32(&sm.p_ready[b][0]), (j / kSBufs) & 1, abort_flag)) &&
                     __all_sync(kFull, mbar_wait(smem_u32(&sm.p_ready[b][1]), (j / kSBufs) & 1, abort_flag));
                if (!ok) break;
            }
            tc_fence_after();
            const uint64_t vd = v_desc0 + static_cast<uint64_t>(s) * (kTileBytes >> 4);
            const uint32_t a_p = tmem + kColS + b * kTile;  // bf16 P: half h in columns [64h, 64h+32)
            if (elect_one()) {
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
        }
    } else if (warp < 8) {
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
            }
        }
        for (int j = 1; j < my_tiles && ok; ++j) {
            const int t = t_begin + j, b = j % kSBufs;
            const uint32_t s_addr = lane_addr + kColS + b * kTile + half * 64;
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
            // A parity wait cannot tell phase j-1 from phase j-3: a thread that skipped phases could
            // sail through a later wait while the product it needs is still running.  So every tile
            // observes the previous tile's o_done, here at the latest (by now it has long completed).
            if (!__all_sync(kFull, saw_o_done)) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[half]), (j - 1) & 1, abort_flag));
                if (!ok) break;
            }
            tc_fence_before();
            mbar_arrive(smem_u32(&sm.p_ready[b][half]));
        }

        if (preloaded) tmem_wait_ld();  // only when the loop was left early: no load may outlive the TMEM allocation
        // ---- epilogue: merge the two halves and write each row's 16-bit values straight from registers ----
        for (int h = 0; h < 2 && ok; ++h)
            ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[h]), (my_tiles - 1) & 1, abort_flag));
        const bool direct = p.splits == 1;
        if (ok) {
            tc_fence_after();
            sm.xm[half][wt] = m_run;
            sm.xl[half][wt] = l_run;
            mbar_arrive(smem_u32(&sm.fin));
            ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.fin), 0, abort_flag));
        }
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
    }

    // ---- teardown -------------------------------------------------------------------------------
    tc_fence_before();
    __syncthreads();
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

}  // namespace

cudaError_t tree_attention_halves_opt_in() {
    static_assert(sizeof(Smem) <= 232448, "exceeds the 227 KB of shared memory a CTA may opt in to");
    return cudaFuncSetAttribute(tree_attention_halves_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                static_cast<int>(sizeof(Smem)));
}

cudaError_t launch_tree_attention_halves(dim3 grid, const CUtensorMap& map_q, const CUtensorMap& map_kc, const CUtensorMap& map_vc,
                                         const CUtensorMap& map_kt, const CUtensorMap& map_vt, const KernelParams& p,
                                         cudaStream_t st) {
    return launch_pdl(tree_attention_halves_kernel, grid, dim3(kThreads), sizeof(Smem), st, map_q, map_kc, map_vc, map_kt, map_vt, p);
}

}  // namespace ddtree

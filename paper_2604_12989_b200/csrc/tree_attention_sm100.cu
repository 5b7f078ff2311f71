// bf16 tree attention for sm_100a: split-KV flash-decoding with TMA-staged K/V tiles and tcgen05
// MMAs accumulating in tensor memory (Section 4.4: every tree row attends to the cached prefix
// and, inside the tree, to the rows named by its ancestor mask).
//
// Rows of one KV head are the (node, g) pairs of its G = Hq/Hkv query heads, row = node*G + g, so
// that budget x G rows share each K/V tile and QK^T / PV are dense 128x128x128 contractions.
//
// One CTA = one (request, KV head, pair of 128-row tiles A and B, KV split).  Warp roles:
//   warps 0-3  softmax of row tile A: one thread per row (TMEM lane = row), all 128 key columns of a
//              KV tile, read from tensor memory 64 at a time
//   warps 4-7  softmax of row tile B, the same
//   warp 8     TMA producer: Q_A, Q_B once, then one ring of K and V tiles (K_0, V_0, K_1, V_1, ...)
//   warp 9     MMA issuer; owns the TMEM allocation.  Per KV tile j it issues, for A and then for B,
//              O_X += P_X V_j followed by S_X = Q_X K_{j+1}^T: the products of one row tile run while
//              the other row tile's threads exponentiate, so that the tensor pipe and the
//              exponential unit, which cost the same per tile at head dim 128, overlap
//   warp 10    clears the rows of a staged V tile that belong to no visible key (the ragged end of a
//              prefix, tree rows past n_rows): their probabilities are zero, but 0 x NaN is not
// Tensor memory: S_A, S_B (fp32 scores, 128 columns each; the bf16 probabilities overwrite the first
// 64 columns of their own scores), O_A, O_B (128 columns each): all 512 columns.
// A last row tile of at most 16 rows (the root's G rows of a tree of 2^k nodes) is a CTA of its own
// with the roles of rows and keys swapped: see tail_tile_cta.
// The ancestor bitmask is applied only on tree tiles; prefix tiles need at most a length test on
// the request's last tile.  Each split writes its normalised rows (fp16) with their reference maximum
// and sum; a combine kernel merges them by log-sum-exp.  Every wait is bounded: when one gives up, the
// CTA raises a flag in the device status word, drains its copies and leaves without touching its outputs.
#include "sm100_attention.cuh"
#include <algorithm>
#include <atomic>
#include <cmath>
#include <mutex>
#include <type_traits>
#include <unordered_map>
#include <vector>

namespace ddtree {
namespace {
using namespace sm100;

constexpr int kRing = 5;              // K/V tiles in flight: K_j in slot 2j % 5, V_j in slot (2j+1) % 5
constexpr int kProducerWarp = 8, kMmaWarp = 9, kFixWarp = 10;
constexpr int kThreads = 384;         // warps 0-3 / 4-7: softmax A / B; 8: producer; 9: MMA; 10: V clean-up; 11: idle
constexpr uint32_t kColS = 0;         // S_X at column 128 X; P_X (bf16 pairs) in its first 64 columns
constexpr uint32_t kColO = 256;       // O_X at column 256 + 128 X
constexpr int kRegsSoftmax = 208, kRegsOther = 88;  // 256 x 208 + 128 x 88 = 384 x 168 registers

struct Smem {
    uint8_t q[2][kTileBytes];        // row tiles A and B
    uint8_t kv[kRing][kTileBytes];
    uint64_t q_full[2], kv_full[kRing], kv_free[kRing], v_fix[kRing];
    uint64_t s_full[2], p_half[2], p_ready[2], o_half[2], o_final[2];
    uint64_t q_rot[2], k_rot[kRing];  // rotary variant: Q tile rotated by its row tile's threads, tree K tile by the relay warp
    uint32_t tmem_base;
    uint32_t abort;
};


// ---- short last row tile ----------------------------------------------------------------------
// A tree of B = 2^k nodes plus the root leaves G rows over for a last row tile of their own; run
// through the main path, that tile would cost as much as a full one.  With so few rows the roles of
// rows and keys are swapped for the scores: S^T = K Q^T puts the 128 keys of a tile on the TMEM lanes
// and the (at most 16) rows on the columns, so a thread exponentiates 16 values per tile instead of
// 128, keeps its own partial row sums, and the tile costs little more than the copy of its K/V.  The
// second product is swapped as well: O^T += V^T P^T with the V tile as the 128-row (MN-major) operand
// and P^T, 16 rows x 128 keys written to shared memory by the key threads, as the narrow one; O^T
// has the head dimension on the lanes and one column per row.  A row's reference maximum is set by
// an exact reduction over the key threads on the first tile and whenever an exponential exceeds
// 2^24; otherwise the threads only meet at one barrier per tile.  Two groups of 128 key threads take
// alternate tiles, each with its own reference maxima, sums and O^T, merged at the end.  The CTA walks
// its KV split of the request and writes the output itself, or its normalised partial rows when the
// short tile's KV range is split.  Measured: ~1200 cycles per KV tile; the tensor pipe is the limit
// (16 instructions per tile that each stream a 4 KB operand from shared memory).
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
    uint64_t v_fix[kTailVStages];
    // One barrier per buffer, each watched by one key group only: a parity wait must see every phase in turn.
    uint64_t s_full[kTailSBufs], p_ready[2][2], o_done[2][2];
    float red[2][4][kTailRows];  // [group][warp]: row maxima inside the loop, row sums at the end
    float mref[2][kTailRows];    // the groups' reference maxima, exchanged at the end
    uint32_t tmem_base;
    uint32_t abort;
    uint32_t key_fail[2];  // per group: a key thread's wait gave up (written before, read after a barrier of the group)
};

__device__ __noinline__ void tail_tile_cta(const CUtensorMap* map_qt, const CUtensorMap* map_kc, const CUtensorMap* map_vc,
                                              const CUtensorMap* map_kt, const CUtensorMap* map_vt, const KernelParams& p,
                                              uint8_t* smem_raw, int kvh, int r, int n, int split) {
    TailSmem& sm = *reinterpret_cast<TailSmem*>(smem_raw);
    const int rt = p.full_tiles;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int rows = min(n * p.G - rt * kTile, kTailRows);  // valid rows of this tile (> 0: checked by the caller)
    const int p0 = p.cu_prefix[r], P = p.cu_prefix[r + 1] - p0;
    const int prefix_tiles = (P + kTile - 1) / kTile, tree_tiles = (n + kTile - 1) / kTile;
    const int tiles = prefix_tiles + tree_tiles;
    const int per = (tiles + p.tail_splits - 1) / p.tail_splits;
    const int t_begin = split * per;
    const int my_tiles = max(0, min(tiles, t_begin + per) - t_begin);
    const bool direct = p.tail_splits == 1;
    const size_t part_row0 = ((static_cast<size_t>(split) * p.R + r) * p.Hkv + kvh) * p.rows_pad + rt * kTile;
    if (my_tiles == 0) {  // this split has nothing to do for this request: publish empty partials
        if (tid < rows) p.part_ml[part_row0 + tid] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }

    volatile uint32_t* abort_flag = &sm.abort;
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
        for (int s = 0; s < kTailVStages; ++s) {
            mbar_init(smem_u32(&sm.v_full[s]), 1);
            mbar_init(smem_u32(&sm.v_free[s]), 1);
            mbar_init(smem_u32(&sm.v_fix[s]), 1);
        }
        for (int b = 0; b < kTailSBufs; ++b) mbar_init(smem_u32(&sm.s_full[b]), 1);
        for (int b = 0; b < 4; ++b) { mbar_init(smem_u32(&sm.p_ready[0][0]) + 8 * b, 1); mbar_init(smem_u32(&sm.o_done[0][0]) + 8 * b, 1); }
        sm.abort = 0;
        sm.key_fail[0] = 0;
        sm.key_fail[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
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
        fence_async_smem();
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
    } else if (warp == kFixWarp) {
        // Every staged V tile passes through this warp on its way to the MMA warp: rows that no row may see
        // (ragged end of the prefix, tree rows past n_rows) are cleared before the product reads them; their
        // probabilities are zero, but 0 x NaN is not.  The copies run tiles ahead, so the relay costs nothing.
        for (int j = 0; j < my_tiles; ++j) {
            const int s = j % kTailVStages;
            if (!__all_sync(kFull, mbar_wait(smem_u32(&sm.v_full[s]), (j / kTailVStages) & 1, abort_flag))) break;
            const int first = keys_in_tile(t_begin + j, prefix_tiles, P, n);
            if (first < kTile) clear_v_rows(sm.v[s], first, lane);
            if (lane == 0) mbar_arrive(smem_u32(&sm.v_fix[s]));
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
        for (int j = 0; j < my_tiles && ok; ++j) {
            // One burst per tile: O_g^T += V_j^T P_j^T, then the scores of tile j+4 into the S^T buffer the key
            // threads have just read.  Every instruction streams a 128-row operand (4 KB) from shared
            // memory, which takes the tensor pipe ~50 cycles whatever the other extent, so a tile costs it
            // ~850 cycles; the barriers are tested together beforehand to keep it from draining.
            const int s = j % kTailVStages, g = j & 1, b = (j >> 1) & 1;  // key group and its P^T buffer
            const bool more = j + kTailSBufs < my_tiles;
            const bool k_ok = !more || mbar_test(smem_u32(&sm.k_full[(j + kTailSBufs) % kTailKStages]), ((j + kTailSBufs) / kTailKStages) & 1);
            const bool ready = mbar_test(smem_u32(&sm.v_fix[s]), (j / kTailVStages) & 1) & k_ok &
                               mbar_test(smem_u32(&sm.p_ready[g][b]), (j >> 2) & 1);
            if (!__all_sync(kFull, ready)) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.v_fix[s]), (j / kTailVStages) & 1, abort_flag)) &&
                     (!more || wait_k(j + kTailSBufs)) &&
                     __all_sync(kFull, mbar_wait(smem_u32(&sm.p_ready[g][b]), (j >> 2) & 1, abort_flag));
                if (!ok) break;
            }
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
        }
    } else if (warp < 8) {
        // ---- key threads: two groups of 128 (warps 0-3: even tiles, warps 4-7: odd tiles).  Thread c of a
        //      group owns key c of its tiles and head-dim element c of the group's O^T.  A group has its own
        //      reference maxima, sums and O^T: the groups never talk inside the loop and are merged at the
        //      end like two KV splits. ------------------------------------------------------------------
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
            fence_async_smem();
        };
        // completion of the product of this group's q-th tile (it read P^T[q % 2] and added to the group's O^T)
        auto wait_pv = [&](int q) {
            return __all_sync(kFull, mbar_wait(smem_u32(&sm.o_done[g][q & 1]), (q >> 1) & 1, abort_flag));
        };
        bool failed = false;
        for (int q = 0; q < my_count; ++q) {
            const int j = 2 * q + g, t = t_begin + j, b = q & 1, sb = j % kTailSBufs;
            bool ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.s_full[sb]), (j / kTailSBufs) & 1, abort_flag));
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
            float x[kTailRows], pv[kTailRows];
            bool need = false;
#pragma unroll
            for (int i = 0; i < kTailRows; ++i) {
                x[i] = ((vis >> i) & 1u) ? __uint_as_float(sv[i]) * p.scale_log2 : -CUDART_INF_F;
                pv[i] = ex2(x[i] - (mref[i] == -CUDART_INF_F ? 0.f : mref[i]));
                if (i < rows) need |= mref[i] == -CUDART_INF_F || !(pv[i] < 16777216.f);
            }
            // P^T[b] was read by the product of this group's tile q-2
            if (ok && q > 1) ok = wait_pv(q - 2);
            store_p(b, pv);
            // A wait that gave up joins the vote, and the flag it left is read only after the barrier: every
            // thread of the group takes the same way out (a thread missing at a later barrier would hang the others).
            if (!ok) sm.key_fail[g] = 1;
            const bool slow = bar_keys_or(g, need || !ok);
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
        }

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
                        if (direct) {
                            const int grow = rt * kTile + i, node = grow / p.G;
                            const size_t head_row = (static_cast<size_t>(r) * p.N + node) * p.Hq + kvh * p.G + grow % p.G;
                            p.out[head_row * kTile + c] = __float2bfloat16_rn(o);
                            if (c == 0 && p.lse) p.lse[head_row] = (m_row + log2f(l_row)) / kLog2e;
                        } else {
                            p.part_o[(part_row0 + i) * kTile + c] = __float2half_rn(o);
                            if (c == 0) p.part_ml[part_row0 + i] = make_float2(m_row, l_row);
                        }
                    }
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

// ---- main path: softmax of one KV tile by one thread (row) ----------------------------------------
// Visibility of the 128 keys of tile t to a row: vis[w] has bit c set iff key 32 w + c is visible.
// Returns true when all 128 are (no masking needed).
__device__ __forceinline__ bool tile_visibility(uint32_t (&vis)[4], int t, int prefix_tiles, int P, int W, bool valid,
                                                const uint32_t* mrow) {
    bool all_visible = false;
    if (!valid) {
#pragma unroll
        for (int w = 0; w < 4; ++w) vis[w] = 0u;
    } else if (t < prefix_tiles) {
        const int left = P - t * kTile;  // keys of this request in the tile
        all_visible = left >= kTile;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const int lw = left - 32 * w;
            vis[w] = lw >= 32 ? kFull : (lw <= 0 ? 0u : ((1u << lw) - 1u));
        }
    } else {
        const int w0 = (t - prefix_tiles) * 4;
#pragma unroll
        for (int w = 0; w < 4; ++w) vis[w] = w0 + w < W ? mrow[w0 + w] : 0u;
    }
    return all_visible;
}

// Rotary encoding of one row of a staged Q or K tile (two 64-wide halves of 128 rows x 128 bytes, 16-byte chunks
// swizzled with the row index): pair (j, j + 64) is rotated by the angle whose (cos, sin) is tab[j], in float32,
// and rounded back to bf16 in place.
__device__ __forceinline__ void rotate_row(uint8_t* tile, int row, const float2* __restrict__ tab) {
#pragma unroll 2
    for (int c = 0; c < 8; ++c) {
        uint8_t* lo_p = tile + row * 128 + ((c ^ (row & 7)) << 4);
        uint4 lo = *reinterpret_cast<const uint4*>(lo_p), hi = *reinterpret_cast<const uint4*>(lo_p + kHalfBytes);
        __nv_bfloat16* xe = reinterpret_cast<__nv_bfloat16*>(&lo);
        __nv_bfloat16* ye = reinterpret_cast<__nv_bfloat16*>(&hi);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
            const float2 cs = __ldg(tab + c * 8 + e);
            const float x = __bfloat162float(xe[e]), y = __bfloat162float(ye[e]);
            xe[e] = __float2bfloat16_rn(x * cs.x - y * cs.y);
            ye[e] = __float2bfloat16_rn(y * cs.x + x * cs.y);
        }
        *reinterpret_cast<uint4*>(lo_p) = lo;
        *reinterpret_cast<uint4*>(lo_p + kHalfBytes) = hi;
    }
}
// The table row of tree node `node` of request r (its depth = its position minus the root's).
__device__ __forceinline__ const float2* rope_row(const KernelParams& p, int r, int node) {
    const int32_t* pos = p.position_ids + static_cast<size_t>(r) * p.N;
    const int depth = min(max(pos[node] - pos[0], 0), kRopeDepths - 1);
    return p.rope_table + (static_cast<size_t>(r) * kRopeDepths + depth) * 64;
}

template <bool kTail, bool kRope>
__global__ void __launch_bounds__(kThreads, 1)
tree_attention_bf16_kernel(const __grid_constant__ CUtensorMap map_q, const __grid_constant__ CUtensorMap map_kc,
                           const __grid_constant__ CUtensorMap map_vc, const __grid_constant__ CUtensorMap map_kt,
                           const __grid_constant__ CUtensorMap map_vt, const __grid_constant__ CUtensorMap map_qt,
                           const __grid_constant__ KernelParams p) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>(smem_raw);
    if (smem_u32(smem_raw) & 1023u) {  // the 128-byte swizzle needs 1024-byte aligned tiles
        if (threadIdx.x == 0) atomicExch(p.status, kErrAlign);
        return;
    }

    // Barriers and descriptor prefetches touch nothing the previous kernel of the stream may still be writing: they
    // run before the wait for it, and before the first sizes come back from global memory.
    if (threadIdx.x == kProducerWarp * 32) {
        for (int x = 0; x < 2; ++x) {
            mbar_init(smem_u32(&sm.q_full[x]), 1);
            mbar_init(smem_u32(&sm.s_full[x]), 1);
            mbar_init(smem_u32(&sm.p_half[x]), kTile);
            mbar_init(smem_u32(&sm.p_ready[x]), kTile);
            mbar_init(smem_u32(&sm.o_half[x]), 1);
            mbar_init(smem_u32(&sm.o_final[x]), 1);
            mbar_init(smem_u32(&sm.q_rot[x]), kTile);
        }
        for (int s = 0; s < kRing; ++s) {
            mbar_init(smem_u32(&sm.kv_full[s]), 1);
            mbar_init(smem_u32(&sm.kv_free[s]), 1);
            mbar_init(smem_u32(&sm.v_fix[s]), 1);
            mbar_init(smem_u32(&sm.k_rot[s]), 1);
        }
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    } else if (threadIdx.x == kProducerWarp * 32 + 1) {
        prefetch_tensormap(&map_q);
        prefetch_tensormap(&map_kc);
        prefetch_tensormap(&map_vc);
        prefetch_tensormap(&map_kt);
        prefetch_tensormap(&map_vt);
    }
    pdl_wait();               // everything read below may come from the previous kernel of the stream
    const int unit = blockIdx.x % p.units;
    const int kvh = (blockIdx.x / p.units) % p.Hkv;
    const int zr = blockIdx.x / (p.units * p.Hkv);
    const int r = p.ordered ? p.order[zr] : zr;
    const int n = min(p.n_rows[r], p.N);
    const int rows_total = n * p.G;
    if constexpr (kTail) {
        if (unit >= p.pairs * p.splits) {
            if (p.full_tiles * kTile < rows_total)
                tail_tile_cta(&map_qt, &map_kc, &map_vc, &map_kt, &map_vt, p, smem_raw, kvh, r, n, unit - p.pairs * p.splits);
            return;
        }
    }
    const int pair = unit / p.splits, split = unit % p.splits;
    const int rt0 = 2 * pair;
    if (rt0 * kTile >= rows_total) return;  // the whole pair is padding
    const bool has_b = rt0 + 1 < p.full_tiles && (rt0 + 1) * kTile < rows_total;
    const int p0 = p.cu_prefix[r], P = p.cu_prefix[r + 1] - p0;
    const int prefix_tiles = (P + kTile - 1) / kTile, tree_tiles = (n + kTile - 1) / kTile;
    const int tiles = prefix_tiles + tree_tiles;
    const int per = (tiles + p.splits - 1) / p.splits;
    const int t_begin = split * per, t_end = min(tiles, t_begin + per);
    const int my_tiles = max(0, t_end - t_begin);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const size_t part_row0 = ((static_cast<size_t>(split) * p.R + r) * p.Hkv + kvh) * p.rows_pad + rt0 * kTile;

    if (my_tiles == 0) {  // this split has nothing to do for this request: publish empty partials
        if (tid < (has_b ? 2 : 1) * kTile) p.part_ml[part_row0 + tid] = make_float2(-CUDART_INF_F, 0.f);
        return;
    }

    // ---- set-up: the producer initialises the barriers and starts the first copies at once ----
    volatile uint32_t* abort_flag = &sm.abort;
    int issued = 0;  // ring units whose copy was started (producer lane only): unit u = K (u even) or V (u odd) of tile u/2
    const int units_total = 2 * my_tiles;
    auto load_unit = [&](int u) {
        const int t = t_begin + (u >> 1), s = u % kRing;
        const bool in_prefix = t < prefix_tiles;
        const int row = in_prefix ? p0 + t * kTile : r * p.N + (t - prefix_tiles) * kTile;
        const CUtensorMap* map = (u & 1) ? (in_prefix ? &map_vc : &map_vt) : (in_prefix ? &map_kc : &map_kt);
        mbar_expect_tx(smem_u32(&sm.kv_full[s]), kTileBytes);
        for (int h = 0; h < 2; ++h)
            tma_load_3d(smem_u32(sm.kv[s]) + h * kHalfBytes, map, smem_u32(&sm.kv_full[s]), h * 64, kvh, row);
    };
    if (warp == kProducerWarp) {
        // the first copies leave from seven lanes at once (one lane issuing fourteen copies takes ~0.4 us): Q_A and
        // the first K tile (the first product needs both), Q_B, then the rest of the ring
        const int nodes_per_tile = kTile / p.G;
        if (lane == 0 || (lane == 2 && has_b)) {
            const int x = lane >> 1;
            mbar_expect_tx(smem_u32(&sm.q_full[x]), kTileBytes);
            for (int h = 0; h < 2; ++h)
                tma_load_4d(smem_u32(sm.q[x]) + h * kHalfBytes, &map_q, smem_u32(&sm.q_full[x]), h * 64, 0, kvh,
                            r * p.N + (rt0 + x) * nodes_per_tile);
        } else if (lane == 1) {
            load_unit(0);
        } else if (lane >= 3 && lane < 2 + kRing && lane - 2 < units_total) {
            load_unit(lane - 2);
        }
        issued = min(kRing, units_total);
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

    if (warp >= 8) {
        regs_dec<kRegsOther>();
        if (warp == kProducerWarp) {
            // ---- TMA producer: a slot is free again when the product that read it last has completed ----
            if (lane == 0) {
                while (issued < units_total) {
                    if (!mbar_wait(smem_u32(&sm.kv_free[issued % kRing]), ((issued / kRing) - 1) & 1, abort_flag)) break;
                    load_unit(issued++);
                }
            }
        } else if (warp == kFixWarp) {
            // ---- V clean-up: every staged V tile passes through this warp on its way to the MMA warp; rows
            //      that no row may see are cleared (see clear_v_rows).  The copies run tiles ahead of the
            //      products, so the relay is off the critical path.  The warp watches the arrival of every
            //      ring unit in order, K tiles included: a parity wait only tells a phase from its neighbour,
            //      so a waiter that skipped the K tile's phase of a slot could take that phase still being
            //      open for the completion of the V tile's phase after it. ----
            for (int u = 0; u < units_total; ++u) {
                const int s = u % kRing;
                if (!__all_sync(kFull, mbar_wait(smem_u32(&sm.kv_full[s]), (u / kRing) & 1, abort_flag))) break;
                if (u & 1) {
                    const int first = keys_in_tile(t_begin + (u >> 1), prefix_tiles, P, n);
                    if (first < kTile) clear_v_rows(sm.kv[s], first, lane);
                    if (lane == 0) mbar_arrive(smem_u32(&sm.v_fix[s]));
                } else if (kRope && t_begin + (u >> 1) >= prefix_tiles) {
                    // a tile of this round's tree keys: rotate its rows to their positions (cached keys were
                    // rotated when they were produced); rows past the tree are left as they are (masked anyway)
                    const int node0 = (t_begin + (u >> 1) - prefix_tiles) * kTile;
                    for (int row = lane; row < kTile; row += 32)
                        if (node0 + row < n) rotate_row(sm.kv[s], row, rope_row(p, r, node0 + row));
                    fence_async_smem();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sm.k_rot[s]));
                }
            }
        } else if (warp == kMmaWarp) {
            // ---- MMA issuer: the whole warp walks the loop (so that addresses live in uniform registers)
            //      and one elected lane issues ----
            constexpr uint32_t idesc_qk = instr_desc(kTile, false);
            constexpr uint32_t idesc_pv = instr_desc(kTile, true);
            constexpr uint64_t kSlot = kTileBytes >> 4;
            const uint64_t q_desc0 = smem_desc(smem_u32(sm.q[0]), 16);
            const uint64_t k_desc0 = smem_desc(smem_u32(sm.kv[0]), 16);
            const uint64_t v_desc0 = smem_desc(smem_u32(sm.kv[0]), kHalfBytes);
            // S_X = Q_X K_j^T: 16 head-dim elements (32 bytes) per instruction; the second 64-wide half of the
            // tiles sits 16 KB further.  Called by the elected lane only.
            auto issue_qk = [&](int x, int j) {
                const uint64_t kd = k_desc0 + static_cast<uint64_t>((2 * j) % kRing) * kSlot;
                const uint64_t qd = q_desc0 + static_cast<uint64_t>(x) * kSlot;
                const uint32_t d_s = tmem + kColS + x * kTile;
                umma_ss<false>(d_s, qd, kd, idesc_qk);
                umma_ss<true>(d_s, qd + 2, kd + 2, idesc_qk);
                umma_ss<true>(d_s, qd + 4, kd + 4, idesc_qk);
                umma_ss<true>(d_s, qd + 6, kd + 6, idesc_qk);
                umma_ss<true>(d_s, qd + 1024, kd + 1024, idesc_qk);
                umma_ss<true>(d_s, qd + 1026, kd + 1026, idesc_qk);
                umma_ss<true>(d_s, qd + 1028, kd + 1028, idesc_qk);
                umma_ss<true>(d_s, qd + 1030, kd + 1030, idesc_qk);
            };
            // O_X += P_X V_j, keys [64 h, 64 h + 64) of the tile: 16 keys (16 rows of 128 bytes of V, 8 columns of
            // bf16 pairs of P) per instruction
            auto issue_pv = [&](int x, int j, int h) {
                const uint64_t vd = v_desc0 + static_cast<uint64_t>((2 * j + 1) % kRing) * kSlot + h * 512;
                const uint32_t a_p = tmem + kColS + x * kTile + h * 32, d_o = tmem + kColO + x * kTile;
                if (j > 0 || h) umma_ts<true>(d_o, a_p, vd, idesc_pv);
                else umma_ts<false>(d_o, a_p, vd, idesc_pv);
                umma_ts<true>(d_o, a_p + 8, vd + 128, idesc_pv);
                umma_ts<true>(d_o, a_p + 16, vd + 256, idesc_pv);
                umma_ts<true>(d_o, a_p + 24, vd + 384, idesc_pv);
            };
            auto wait_bar = [&](uint64_t* bar, uint32_t parity) {
                return __all_sync(kFull, mbar_wait(smem_u32(bar), parity, abort_flag));
            };
            auto wait_unit = [&](int u) { return wait_bar(&sm.kv_full[u % kRing], (u / kRing) & 1); };
            const int last_x = has_b ? 1 : 0;  // the row tile whose products release the K/V slots
            uint32_t rot_phase = 0;  // rotary variant: per ring slot, parity of its next rotated tree K tile
            // K tile of ring unit u staged (and, for a tile of tree keys in the rotary variant, rotated)
            auto wait_k = [&](int u) {
                bool good = wait_unit(u);
                if (kRope && good && t_begin + (u >> 1) >= prefix_tiles) {
                    const int s = u % kRing;
                    good = wait_bar(&sm.k_rot[s], (rot_phase >> s) & 1);
                    rot_phase ^= 1u << s;
                }
                return good;
            };
            bool ok = wait_bar(kRope ? &sm.q_rot[0] : &sm.q_full[0], 0) && wait_k(0);
            if (ok) {
                tc_fence_after();
                if (elect_one()) { issue_qk(0, 0); tc_commit(smem_u32(&sm.s_full[0])); if (!has_b) tc_commit(smem_u32(&sm.kv_free[0])); }
                __syncwarp();
            }
            if (ok && has_b) {
                ok = wait_bar(kRope ? &sm.q_rot[1] : &sm.q_full[1], 0);
                if (ok) {
                    tc_fence_after();
                    if (elect_one()) { issue_qk(1, 0); tc_commit(smem_u32(&sm.s_full[1])); tc_commit(smem_u32(&sm.kv_free[0])); }
                    __syncwarp();
                }
            }
            for (int j = 0; j < my_tiles && ok; ++j) {
                const bool more = j + 1 < my_tiles;
                const int uv = 2 * j + 1, sv_slot = uv % kRing;
                for (int x = 0; x <= last_x && ok; ++x) {
                    if (x == 0) {
                        // V_j staged and passed on by the clean-up warp (a slot holds K and V tiles in turn: every
                        // other use is a V tile), K_{j+1} staged: copies run far ahead, these rarely wait
                        ok = wait_bar(&sm.v_fix[sv_slot], ((uv / kRing) >> 1) & 1) && (!more || wait_k(uv + 1));
                        if (!ok) break;
                    }
                    // the probabilities arrive in two halves of 64 keys: the product over the first half runs
                    // while the row tile's threads still exponentiate the second
                    ok = wait_bar(&sm.p_half[x], j & 1);
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
                        issue_pv(x, j, 0);
                        tc_commit(smem_u32(&sm.o_half[x]));
                    }
                    __syncwarp();
                    ok = wait_bar(&sm.p_ready[x], j & 1);
                    if (!ok) break;
                    tc_fence_after();
                    if (elect_one()) {
                        issue_pv(x, j, 1);
                        if (x == last_x) tc_commit(smem_u32(&sm.kv_free[sv_slot]));
                        if (more) {
                            issue_qk(x, j + 1);
                            tc_commit(smem_u32(&sm.s_full[x]));
                            if (x == last_x) tc_commit(smem_u32(&sm.kv_free[(uv + 1) % kRing]));
                        } else {
                            tc_commit(smem_u32(&sm.o_final[x]));
                        }
                    }
                    __syncwarp();
                }
            }
        }
    } else {
        regs_inc<kRegsSoftmax>();
        // ---- softmax: thread `row` of group X owns row `row` of row tile rt0 + X: all 128 scores of every KV
        //      tile, its own reference maximum and sum; nobody else ever touches that row ----
        const int x = warp >> 2, row = tid & (kTile - 1);
        if (x == 0 || has_b) {
            const int grow = (rt0 + x) * kTile + row;   // row among this KV head's rows
            const int node = grow / p.G;
            const bool valid = node < n;
            const uint32_t* mrow = p.anc_mask + (static_cast<size_t>(r) * p.N + (valid ? node : 0)) * p.W;
            const uint32_t lane_addr = tmem + (static_cast<uint32_t>((warp & 3) * 32) << 16);
            const uint32_t s_addr = lane_addr + kColS + x * kTile;
            const uint32_t o_addr = lane_addr + kColO + x * kTile;
            float m_run = -CUDART_INF_F, l_run = 0.f;  // reference maximum (scaled log2 units; -inf: no key seen yet), sum
            bool ok = true;
            if constexpr (kRope) {
                // rotary variant: every thread rotates its own query row in the staged tile before the first product
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.q_full[x]), 0, abort_flag));
                if (ok && valid) rotate_row(sm.q[x], row, rope_row(p, r, node));
                fence_async_smem();
                mbar_arrive(smem_u32(&sm.q_rot[x]));
            }
            // A tile's scores come from tensor memory one half (64 columns) at a time: few registers are live (with
            // all 128 scores of a row in registers the compiler has no room to keep exponentials in flight), and
            // there are only two round trips per tile (a load in flight holds the warp back; the other row tile's
            // warp on the same sub-partition fills the gap).
            uint32_t sc[64], pk[32];
            // Per half (64 keys) of a tile, an optimistic pass: exponentials relative to the reference maximum as it
            // stands.  P keeps its relative precision whatever the reference (bf16 has the exponent range of fp32),
            // so the reference only has to keep the sums away from overflow: it is revisited when a row sum exceeds
            // 2^24 (or is not finite), and for a row that sees its first key.  Then the probabilities go over the
            // scores' own columns and the MMA warp is told.
            for (int j = 0; j < my_tiles && ok; ++j) {
                ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.s_full[x]), j & 1, abort_flag));
                if (!ok) break;  // warp-uniform: the TMEM loads/stores below need the whole warp
                tc_fence_after();
                uint32_t vis[4];
                const bool all_visible = tile_visibility(vis, t_begin + j, prefix_tiles, P, p.W, valid, mrow);
                // the two halves run through the same code (one copy of the unrolled exponent loop: short CTAs
                // pay for every instruction they fetch for the first time)
#pragma unroll 1
                for (int kh = 0; kh < 2; ++kh) {
                    tmem_ld64(sc, s_addr + 64 * kh);
                    const uint32_t vis0 = kh ? vis[2] : vis[0], vis1 = kh ? vis[3] : vis[1];
                    const bool sees = all_visible || (vis0 | vis1) != 0u;
                    tmem_wait_ld();
                    if (!all_visible) { mask32(sc, 0, vis0); mask32(sc, 32, vis1); }
                    float rowsum = exp_pack_64(sc, pk, p.scale_log2, m_run == -CUDART_INF_F ? 0.f : m_run);
                    const bool revisit = m_run == -CUDART_INF_F ? sees : !(rowsum < 16777216.f);
                    if (__any_sync(kFull, revisit)) {
                        // exact maximum of my 64 scores (still in registers); the reference moves only when the
                        // maximum outgrew it by 2^8
                        const float m_tile = max_64(sc) * p.scale_log2;  // -inf if I see no key of this half
                        const bool bump = m_tile > m_run + 8.f;
                        const float alpha = bump ? ex2(m_run - m_tile) : 1.f;
                        if (bump) { l_run *= alpha; m_run = m_tile; }
                        if ((j > 0 || kh) && __any_sync(kFull, bump)) {
                            // O_X holds the sum over everything before this half.  The product of tile j-1 completed
                            // before this tile's scores were announced; the product over this tile's first half is
                            // waited for here.  Then my row is rescaled.
                            if (kh && !__all_sync(kFull, mbar_wait(smem_u32(&sm.o_half[x]), j & 1, abort_flag))) { ok = false; break; }
                            tc_fence_after();
#pragma unroll 1
                            for (int c0 = 0; c0 < 128; c0 += 32) {
                                TMEM_LD32(pk, 0, o_addr + c0);
                                tmem_wait_ld();
#pragma unroll
                                for (int c = 0; c < 32; ++c) pk[c] = __float_as_uint(__uint_as_float(pk[c]) * alpha);
                                TMEM_ST32(o_addr + c0, pk, 0);
                            }
                            tmem_wait_st();
                        }
                        rowsum = exp_pack_64(sc, pk, p.scale_log2, m_run == -CUDART_INF_F ? 0.f : m_run);
                    }
                    TMEM_ST32(s_addr + 32 * kh, pk, 0);
                    l_run += rowsum;
                    tmem_wait_st();
                    tc_fence_before();
                    mbar_arrive(smem_u32(kh ? &sm.p_ready[x] : &sm.p_half[x]));
                }
            }

            // ---- epilogue: each thread normalises its row and writes its 256 contiguous bytes itself: to the
            //      output (bf16) when this CTA saw the whole KV range, else to the split partials (fp16: the rows
            //      are averages of V rows, so fp16's 11 bits are finer than the bf16 rounding of the final output).
            //      (An SM stores ~32 bytes per clock whatever the route: staging the rows for coalesced stores
            //      or for one bulk tensor store was measured and takes the same time.) ----
            if (ok) ok = __all_sync(kFull, mbar_wait(smem_u32(&sm.o_final[x]), 0, abort_flag));
            if (ok) {
                tc_fence_after();
                const bool direct = p.splits == 1;
                const float f = l_run > 0.f ? 1.f / l_run : 0.f;  // rows leave normalised, also as split partials
                uint16_t* dst16;
                if (direct) {
                    dst16 = reinterpret_cast<uint16_t*>(p.out) +
                            ((static_cast<size_t>(r) * p.N + (valid ? node : 0)) * p.Hq + kvh * p.G + grow % p.G) * kTile;
                } else {
                    dst16 = reinterpret_cast<uint16_t*>(p.part_o) + (part_row0 + x * kTile + row) * kTile;
                }
#pragma unroll
                for (int c0 = 0; c0 < 128; c0 += 32) {
                    uint32_t w16[16];
                    TMEM_LD32(sc, 0, o_addr + c0);
                    tmem_wait_ld();
#pragma unroll
                    for (int q = 0; q < 16; ++q) {
                        const float a = __uint_as_float(sc[2 * q]) * f, b = __uint_as_float(sc[2 * q + 1]) * f;
                        if (direct) {
                            const __nv_bfloat162 t2 = __floats2bfloat162_rn(a, b);
                            w16[q] = *reinterpret_cast<const uint32_t*>(&t2);
                        } else {
                            const __half2 t2 = __floats2half2_rn(a, b);
                            w16[q] = *reinterpret_cast<const uint32_t*>(&t2);
                        }
                    }
                    if (valid) {
                        st_global_256(dst16 + c0, w16, 0);
                        st_global_256(dst16 + c0 + 16, w16, 8);
                    }
                }
                if (valid) {
                    if (direct) {
                        if (p.lse) p.lse[(static_cast<size_t>(r) * p.N + node) * p.Hq + kvh * p.G + grow % p.G] = (m_run + log2f(l_run)) / kLog2e;
                    } else {
                        p.part_ml[part_row0 + x * kTile + row] = make_float2(m_run, l_run);
                    }
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
            mbar_wait(smem_u32(&sm.q_full[0]), 0, &scratch);
            if (has_b) mbar_wait(smem_u32(&sm.q_full[1]), 0, &scratch);
            for (int u = max(0, issued - kRing); u < issued; ++u)
                mbar_wait(smem_u32(&sm.kv_full[u % kRing]), (u / kRing) & 1, &scratch);
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
    const int nodes = p.N - p.node0;
    const long long task = static_cast<long long>(blockIdx.x) * 4 + warp;
    if (task >= static_cast<long long>(p.R) * nodes * p.Hq) return;
    const int h = static_cast<int>(task % p.Hq);
    const int node = p.node0 + static_cast<int>((task / p.Hq) % nodes);
    const int r = static_cast<int>(task / (static_cast<long long>(p.Hq) * nodes));
    const int kvh = h / p.G, grow = node * p.G + h % p.G;
    const int splits = (p.tail && grow >= p.full_tiles * kTile) ? p.tail_splits : p.splits;
    if (splits == 1) return;  // written by its CTA directly
    const size_t split_stride = static_cast<size_t>(p.R) * p.Hkv * p.rows_pad;
    const size_t row0 = (static_cast<size_t>(r) * p.Hkv + kvh) * p.rows_pad + grow;
    // One round trip to L2 for everything this row needs: the row count of the request, the (max, sum)
    // pairs and the rows of up to 8 splits are requested together, before any of them is looked at
    // (rows of padding nodes and of empty splits lie inside the buffer; their contents are never used).
    const __half* po = p.part_o + row0 * kTile + lane * 4;
    const int n_r = p.n_rows[r];
    float2 ml = make_float2(-CUDART_INF_F, 0.f);
    if (lane < splits) ml = p.part_ml[lane * split_stride + row0];
    uint2 raw[8];
#pragma unroll
    for (int u = 0; u < 8; ++u)
        raw[u] = u < splits ? *reinterpret_cast<const uint2*>(po + u * split_stride * kTile) : make_uint2(0u, 0u);
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
        if (u < splits) add(u, raw[u]);
    for (int s = 8; s < splits; ++s) add(s, *reinterpret_cast<const uint2*>(po + s * split_stride * kTile));
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

// Rotary variant: (cos, sin) of position x theta^(-2j/128) for every request, every depth a tree row can have and
// the 64 frequency pairs of a head.  The angle is formed and reduced modulo 2 pi in double precision (positions
// reach 10^5, where a float32 angle is off by 10^-2 rad), sine and cosine are taken in float32 on the reduced angle.
struct RopeFreq64 {
    double inv_freq[64];
};
__global__ void rope_table_kernel(const int32_t* __restrict__ position_ids, int N, float2* __restrict__ table,
                                  const __grid_constant__ RopeFreq64 f) {
    pdl_wait();
    const int r = blockIdx.x;
    const double pos0 = static_cast<double>(position_ids[static_cast<size_t>(r) * N]);  // the root's position
    for (int i = threadIdx.x; i < kRopeDepths * 64; i += blockDim.x) {
        const int depth = i >> 6, j = i & 63;
        const double a = (pos0 + depth) * f.inv_freq[j];
        const double turns = rint(a * 0.15915494309189535);
        const double red = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, a));
        float sn, cs;
        sincosf(static_cast<float>(red), &sn, &cs);
        table[(static_cast<size_t>(r) * kRopeDepths + depth) * 64 + j] = make_float2(cs, sn);
    }
}

// A wait that nothing can satisfy: one thread initialises a barrier nobody arrives at, polls it `limit`
// times, gives up and raises the time-out flag in the device status word, exactly as the attention
// kernel's waits do.  The kernel returns normally.  (Self-test of the reporting path: see
// ddtree_selftest_wait_timeout.)
__global__ void wait_timeout_selftest_kernel(uint32_t* status, uint32_t limit) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort;
    pdl_wait();
    if (threadIdx.x == 0) {
        abort = 0;
        mbar_init(smem_u32(&bar), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (!mbar_wait_limit(smem_u32(&bar), 0, &abort, limit)) atomicExch(status, kErrTimeout);
    }
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

constexpr int kSMs = 148;

struct Plan {
    int row_tiles, rows_pad;
    int halves;  // 1: one row tile per CTA (tree_attention_sm100_halves.cu), `splits` KV splits for every row tile
    int full_tiles, pairs, tail;
    int splits, tail_splits, units;
    size_t off_ml, off_rope, total;
};

std::atomic<int> g_path{0};  // 0: chosen by the cost model, 1: two row tiles per CTA, 2: one row tile per CTA

// How the rows and the KV range of a call are spread over CTAs.  A batch that fills the SMs more than once
// runs unsplit, two row tiles per CTA.  Otherwise every CTA is resident at once and the KV range is split so
// that all CTAs finish together; the costs below (cycles, from device time stamps of layers whose K/V come
// from HBM and a sweep of 250 shapes timed on both kernels) are: a CTA of row-tile pairs 15600 + 4100 per
// KV tile, a short-tile CTA 24000 + 1400 per tile, a CTA of one row tile 8000 + 2000 per tile, the merge of
// split partials 9000.  With few tiles per CTA the fixed terms decide, and one row tile per CTA reaches the
// same number of resident CTAs with half the splits (half the partial rows to write and to merge), or with
// none.  On that sweep the choice below is within 0.3 % of the faster kernel on average.
Plan make_plan(const AttnArgs& a, int path) {
    Plan pl;
    pl.row_tiles = (a.N * a.G + kTile - 1) / kTile;
    pl.rows_pad = pl.row_tiles * kTile;
    pl.halves = 0;
    // (the rotary variant runs a short last tile through the main path: one code path rotates)
    pl.tail = (!a.rope && a.N * a.G - (pl.row_tiles - 1) * kTile <= kTailRows) ? 1 : 0;
    pl.full_tiles = pl.row_tiles - pl.tail;
    pl.pairs = (pl.full_tiles + 1) / 2;
    const int groups = a.R * a.Hkv;
    const int max_tiles = (a.max_prefix + kTile - 1) / kTile + (a.N + kTile - 1) / kTile;
    pl.splits = 1;
    pl.tail_splits = 1;
    if (groups * (pl.pairs + pl.tail) < kSMs) {
        const int budget = kSMs / groups;                   // CTAs per (request, KV head)
        const int s_cap = std::max(1, std::min(32, (max_tiles + 1) / 2));  // at least two KV tiles per split
        const int t_cap = std::max(1, std::min(32, (max_tiles + 3) / 4));
        double best = 1e30;
        for (int s = 1; s <= (pl.pairs ? s_cap : 1); ++s) {
            for (int t = 1; t <= (pl.tail ? t_cap : 1); ++t) {
                if (pl.pairs * s + pl.tail * t > budget) break;
                const double cf = pl.pairs ? 15600.0 + 4100.0 * ((max_tiles + s - 1) / s) : 0.0;
                const double ct = pl.tail ? 24000.0 + 1400.0 * ((max_tiles + t - 1) / t) : 0.0;
                const double cost = std::max(cf, ct) + 1.0 * (pl.pairs * s + pl.tail * t);  // ties: fewer CTAs
                if (cost < best) { best = cost; pl.splits = s; pl.tail_splits = t; }
            }
        }
        // one row tile per CTA instead?
        if (!a.rope && path != 1 && groups * pl.row_tiles <= kSMs) {
            const int s = std::max(1, std::min(std::min(32, kSMs / (groups * pl.row_tiles)), (max_tiles + 1) / 2));
            constexpr double kMerge = 9000.0;
            const double cp = best + (pl.splits > 1 || (pl.tail && pl.tail_splits > 1) ? kMerge : 0.0);
            const double ch = 8000.0 + 2000.0 * ((max_tiles + s - 1) / s) + (s > 1 ? kMerge : 0.0);
            // (long loops: in a train of layers at the power cap the two-row-tile kernel holds the higher clock, so
            // the other has to win by more than the sweep's single bursts show)
            const double margin = (max_tiles + s - 1) / s >= 48 ? 0.925 : 0.95;
            if (path == 2 || ch < margin * cp) {
                pl.halves = 1;
                pl.tail = 0;
                pl.full_tiles = pl.row_tiles;
                pl.pairs = 0;
                pl.splits = s;
                pl.tail_splits = 1;
            }
        }
    }
    pl.units = pl.halves ? pl.row_tiles * pl.splits : pl.pairs * pl.splits + pl.tail * pl.tail_splits;
    const int smax = std::max(pl.splits, pl.tail ? pl.tail_splits : 1);
    const size_t rows = static_cast<size_t>(smax) * a.R * a.Hkv * pl.rows_pad;
    pl.off_ml = (rows * kTile * 2 + 255) / 256 * 256;
    pl.off_rope = pl.off_ml + (rows * 8 + 255) / 256 * 256;
    if (smax == 1) { pl.off_ml = 0; pl.off_rope = 0; }
    pl.total = pl.off_rope + (a.rope ? static_cast<size_t>(a.R) * kRopeDepths * 64 * sizeof(float2) : 0);
    if (pl.total < 256) pl.total = 256;
    return pl;
}

}  // namespace

size_t tree_attention_bf16_workspace(const AttnArgs& a, const int32_t*) {
    // one answer for ddtree_tree_attention and ddtree_tree_attention_rope (their plans differ in the short tile)
    // and whichever kernel the cost model or ddtree_tree_attention_set_path picks at launch time
    AttnArgs plain = a, rope = a;
    plain.rope = 0;
    rope.rope = 1;
    return std::max(make_plan(rope, 1).total, std::max(make_plan(plain, 1).total, make_plan(plain, 2).total));
}

int tree_attention_bf16_kernels(const AttnArgs& a) {
    const Plan pl = make_plan(a, g_path.load(std::memory_order_relaxed));
    return 1 + ((pl.splits > 1 || (pl.tail && pl.tail_splits > 1)) ? 1 : 0) + (a.rope ? 1 : 0);
}

void tree_attention_set_path(int path) { g_path.store(path < 0 || path > 2 ? 0 : path, std::memory_order_relaxed); }

int launch_tree_attention_bf16(const AttnArgs& a, const int32_t* cu_prefix_host, void* ws, size_t, cudaStream_t st) {
    const Plan pl = make_plan(a, g_path.load(std::memory_order_relaxed));
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
    p.rows_pad = pl.rows_pad;
    p.full_tiles = pl.full_tiles; p.pairs = pl.pairs; p.splits = pl.splits;
    p.tail = pl.tail; p.tail_splits = pl.tail_splits; p.units = pl.units;
    // the combine kernel visits every row when the pairs are split, else only the short tile's rows
    p.node0 = pl.splits > 1 ? 0 : (pl.full_tiles * kTile) / a.G;
    p.scale_log2 = a.scale * kLog2e;
    p.position_ids = a.position_ids;
    p.rope_table = reinterpret_cast<const float2*>(static_cast<const char*>(ws) + pl.off_rope);
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
            cudaError_t e = cudaFuncSetAttribute(tree_attention_bf16_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                 static_cast<int>(smem_bytes));
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(tree_attention_bf16_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem_bytes));
            if (e == cudaSuccess)
                e = cudaFuncSetAttribute(tree_attention_bf16_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem_bytes));
            if (e == cudaSuccess) e = tree_attention_halves_opt_in();
            if (e != cudaSuccess)
                return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: shared memory opt-in: %s", cudaGetErrorString(e));
            if (dev >= 0 && dev < 64) done[dev] = true;
        }
    }
    const long long ctas = static_cast<long long>(a.R) * a.Hkv * pl.units;
    if (ctas > 0x7fffffffLL) return fail(DDTREE_ERR_UNSUPPORTED, "ddtree_tree_attention: grid too large");
    dim3 grid(static_cast<unsigned>(ctas));
    cudaError_t e = cudaSuccess;
    if (pl.halves) {
        e = launch_tree_attention_halves(dim3(pl.splits, a.Hkv * pl.row_tiles, a.R), mq, mkc, mvc, mkt, mvt, p, st);
    } else if (a.rope) {
        RopeFreq64 f;
        for (int j = 0; j < 64; ++j) f.inv_freq[j] = std::exp2(-(2.0 * j / kTile) * a.rope_log2_theta);
        e = launch_pdl(rope_table_kernel, dim3(a.R), dim3(256), 0, st, a.position_ids,  a.N,
                       reinterpret_cast<float2*>(static_cast<char*>(ws) + pl.off_rope), f);
        if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention_rope: table: %s", cudaGetErrorString(e));
        e = launch_pdl(tree_attention_bf16_kernel<false, true>, grid, dim3(kThreads), smem_bytes, st, mq, mkc, mvc, mkt, mvt, mqt, p);
    } else {
        e = pl.tail
            ? launch_pdl(tree_attention_bf16_kernel<true, false>, grid, dim3(kThreads), smem_bytes, st, mq, mkc, mvc, mkt, mvt, mqt, p)
            : launch_pdl(tree_attention_bf16_kernel<false, false>, grid, dim3(kThreads), smem_bytes, st, mq, mkc, mvc, mkt, mvt, mqt, p);
    }
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: launch: %s", cudaGetErrorString(e));
    if (pl.splits > 1 || (pl.tail && pl.tail_splits > 1)) {
        const long long tasks = static_cast<long long>(a.R) * (a.N - p.node0) * a.Hq;
        e = launch_pdl(combine_kernel, dim3(static_cast<unsigned>((tasks + 3) / 4)), dim3(128), 0, st, p);
        if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: combine: %s", cudaGetErrorString(e));
    }
    return DDTREE_OK;
}

cudaError_t launch_wait_timeout_selftest(uint32_t limit, cudaStream_t st) {
    uint32_t* status = device_status_word();
    if (!status) return cudaErrorUnknown;
    return launch_pdl(wait_timeout_selftest_kernel, dim3(1), dim3(32), 0, st, status, limit);
}

}  // namespace ddtree

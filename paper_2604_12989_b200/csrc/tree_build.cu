// One CTA per request: merge the per-chunk partials of the logits pass into the [L,K] table of
// log-probabilities, run the best-first selection of Algorithm 1 on one warp in shared memory, and
// flatten the selected prefixes into the verifier's inputs (Section 4.4).
//
// Algorithm 1's heap always holds, for every node already selected (and for the root), exactly one
// entry: that node's next unselected child (a "next sibling" push is the parent's next child, a
// "first child" push is the popped node's first child).  The warp therefore keeps one candidate
// score per selected node, cand(u) = sigma(u) + log q_{depth(u)+1}^{(children(u)+1)}, spread over
// its lanes (slot s lives on lane s % 32), and a pop is a warp-wide arg-max instead of a sift
// through a binary heap.  The pop sequence is the same as Algorithm 1's up to the order of equal
// scores.
#include "common.cuh"
#include <math_constants.h>

namespace ddtree {
namespace {

constexpr int kThreads = 512;
constexpr int kWarps = kThreads / 32;
constexpr unsigned kFull = 0xffffffffu;
constexpr int kSlots = 1056;  // >= kMaxN, multiple of 32
constexpr int kMaxHits = 64;

__device__ __forceinline__ unsigned orderable(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// Sorted list of the best entries seen by a warp: lane k holds the k-th best (value, id).
struct WarpTopK {
    float tv;   // this lane's entry
    int ti;
    float thr_v;  // entry of lane K-1 (what a candidate has to beat), never below the floor
    int thr_i;
    float floor_v;  // values below the floor are known not to be among the K best
    __device__ __forceinline__ void init(float floor_value) {
        tv = -CUDART_INF_F; ti = -1;
        floor_v = floor_value; thr_v = floor_value; thr_i = 0x7fffffff;
    }
    // Warp-collective: insert a candidate that beats the threshold.
    __device__ __forceinline__ void insert(float v, int id, int K, int lane) {
        const bool mine_first = beats(tv, ti, v, id);
        const int pos = __popc(__ballot_sync(kFull, mine_first));
        const float upv = __shfl_up_sync(kFull, tv, 1);
        const int upi = __shfl_up_sync(kFull, ti, 1);
        if (lane == pos) { tv = v; ti = id; }
        else if (lane > pos) { tv = upv; ti = upi; }
        thr_v = __shfl_sync(kFull, tv, K - 1);
        thr_i = __shfl_sync(kFull, ti, K - 1);
        if (thr_i < 0) { thr_v = floor_v; thr_i = 0x7fffffff; }  // fewer than K entries so far
    }
    // Warp-collective: every lane offers VN candidates vals[e] with ids id0+e.
    template <int VN>
    __device__ __forceinline__ void offer(const float (&vals)[VN], int id0, int K, int lane) {
        unsigned qual = 0;
#pragma unroll
        for (int e = 0; e < VN; ++e)
            if (beats(vals[e], id0 + e, thr_v, thr_i)) qual |= 1u << e;
        unsigned any = __ballot_sync(kFull, qual != 0);
        while (any) {
            const int src = __ffs(any) - 1;
            any &= any - 1;
            const unsigned qs = __shfl_sync(kFull, qual, src);
            const int ids = __shfl_sync(kFull, id0, src);
#pragma unroll
            for (int e = 0; e < VN; ++e) {
                if ((qs >> e) & 1u) {  // warp-uniform
                    const float v = __shfl_sync(kFull, vals[e], src);
                    if (beats(v, ids + e, thr_v, thr_i)) insert(v, ids + e, K, lane);
                }
            }
        }
    }
};

__device__ __forceinline__ float load_logit(const float* p) { return __ldg(p); }
__device__ __forceinline__ float load_logit(const __nv_bfloat16* p) {
    return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
}

__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(kFull, x, o);
    return x;
}

struct Shared {
    float logq[kMaxL * kMaxK];
    int tok[kMaxL * kMaxK];
    float sigma[kSlots];
    float cand[kSlots];
    short parent[kSlots];   // slot of the parent (selection order), -1 for the root
    short row_of[kSlots];   // slot -> row in level order
    short inv[kSlots];      // row -> slot
    short prow[kSlots];     // row -> parent row
    short fc[kSlots];       // row -> first child row
    short bucket[kSlots];   // slots grouped by depth
    unsigned char depth[kSlots];
    unsigned char rank[kSlots];  // 1-based rank among siblings
    unsigned char cc[kSlots];    // children selected so far
    int hits[kWarps][kMaxHits];   // per warp: threads of the logits pass whose elements are read again
    int wlist[kWarps][kMaxHits];  // per warp: warps of the logits pass whose thread maxima are looked at
    int lvl_cnt[kMaxL + 2];
    int lvl_start[kMaxL + 3];
    int lvl_cur[kMaxL + 2];
    int count;
};

template <typename T>
__global__ void __launch_bounds__(kThreads)
tree_build_kernel(int L, int V, int K, int B, int chunks, const float* __restrict__ pm, const float* __restrict__ ps,
                  const float* __restrict__ tmax, const float* __restrict__ wmax, const T* __restrict__ logits, int64_t row_stride,
                  const int32_t* __restrict__ root_token, const int32_t* __restrict__ prefix_len,
                  int32_t* __restrict__ n_rows, int32_t* __restrict__ node_token, int32_t* __restrict__ node_parent,
                  int32_t* __restrict__ node_depth, int32_t* __restrict__ position_ids,
                  uint32_t* __restrict__ anc_mask, int32_t* __restrict__ first_child,
                  int32_t* __restrict__ child_count, float* __restrict__ node_logprob,
                  int32_t* __restrict__ topk_token, float* __restrict__ topk_logprob) {
    __shared__ Shared sh;
    const int r = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int N = B + 1, W = (N + 31) / 32;

    pdl_wait();
    // ---- 1. merge chunk partials: one warp per draft position ---------------------------------
    for (int i = warp; i < L; i += kWarps) {
        const size_t row = static_cast<size_t>(r) * L + i;
        const float* m_c = pm + row * chunks;
        const float* s_c = ps + row * chunks;
        float M = -CUDART_INF_F;
        for (int c = lane; c < chunks; c += 32) M = fmaxf(M, m_c[c]);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) M = fmaxf(M, __shfl_xor_sync(kFull, M, o));
        double S = 0.0;
        for (int c = lane; c < chunks; c += 32)
            S += static_cast<double>(s_c[c]) * exp(static_cast<double>(m_c[c]) - static_cast<double>(M));
        S = warp_sum(S);
        const double lse = static_cast<double>(M) + log(S);

        // K best elements of the row, (value desc, id asc); lane k ends up with rank k+1.
        // The logits pass left the maximum of every warp's 1024 and every thread's 32 elements.  The
        // K-th largest of the 32 lane-wise maxima over the warp maxima is reached by at least K warps,
        // hence by at least K elements: only threads whose maximum reaches it can hold one of the K
        // best, and there are about K of them.  Their elements are read again and inserted into a
        // sorted warp list.
        const int n_w = chunks * (kTopkThreads / 32);
        const float* wm = wmax + row * n_w;
        const float* tm = tmax + row * n_w * 32;
        float lm = -CUDART_INF_F;
        for (int j = lane; j < n_w; j += 32) lm = fmaxf(lm, wm[j]);
        float tau;
        {
            const unsigned key = orderable(lm);
            int above = 0;
#pragma unroll
            for (int o = 1; o < 32; ++o) above += __shfl_xor_sync(kFull, key, o) > key ? 1 : 0;
            const unsigned kth = __reduce_min_sync(kFull, above < K ? key : 0xffffffffu);
            const unsigned u = (kth & 0x80000000u) ? (kth & 0x7fffffffu) : ~kth;
            tau = fmaxf(__uint_as_float(u), -3.0e38f);  // fewer than K elements in the row: take them all
        }
        WarpTopK top;
        top.init(tau);
        constexpr int VN = 16 / sizeof(T);               // elements per 16-byte vector
        constexpr int NV = kTopkChunk / kTopkThreads / VN;  // vectors per thread of a tile
        const T* x = logits + static_cast<int64_t>(row) * row_stride;
        int* hits = sh.hits[warp];
        int n_hits = 0;
        // up to 4 listed threads per round: lane l fetches vector l%8 of listed thread l/8
        auto flush = [&]() {
            for (int h0 = 0; h0 < n_hits; h0 += 4) {
                const int q = h0 + (lane >> 3), v = lane & 7;
                float vals[VN];
#pragma unroll
                for (int e = 0; e < VN; ++e) vals[e] = -CUDART_INF_F;
                int id0 = 0;
                if (q < n_hits && v < NV) {
                    const int j = hits[q];
                    id0 = (j / kTopkThreads) * kTopkChunk + (v * kTopkThreads + j % kTopkThreads) * VN;
#pragma unroll
                    for (int e = 0; e < VN; ++e)
                        if (id0 + e < V) vals[e] = load_logit(x + id0 + e);
                }
                top.offer<VN>(vals, id0, K, lane);
            }
            n_hits = 0;
        };
        // threads of listed warps whose maximum reaches tau go to the hit list
        int* wlist = sh.wlist[warp];
        int n_wl = 0;
        auto scan_warps = [&]() {
            for (int g = 0; g < n_wl; g += 4) {
                float t4[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) t4[q] = g + q < n_wl ? tm[wlist[g + q] * 32 + lane] : -CUDART_INF_F;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const bool hit = t4[q] >= tau;
                    const unsigned mask = __ballot_sync(kFull, hit);
                    if (!mask) continue;
                    if (n_hits + __popc(mask) > kMaxHits) flush();
                    if (hit) hits[n_hits + __popc(mask & ((1u << lane) - 1u))] = wlist[g + q] * 32 + lane;
                    n_hits += __popc(mask);
                    __syncwarp();
                }
            }
            n_wl = 0;
        };
        for (int j0 = 0; j0 < n_w; j0 += 32) {
            const int j = j0 + lane;
            const bool hit = j < n_w && wm[j] >= tau;
            const unsigned mask = __ballot_sync(kFull, hit);
            if (!mask) continue;
            if (n_wl + __popc(mask) > kMaxHits) scan_warps();
            if (hit) wlist[n_wl + __popc(mask & ((1u << lane) - 1u))] = j;
            n_wl += __popc(mask);
            __syncwarp();
        }
        scan_warps();
        flush();
        const float tv = top.tv;
        const int ti = top.ti;
        if (lane < K) {
            const float lq = static_cast<float>(static_cast<double>(tv) - lse);
            sh.logq[i * K + lane] = lq;
            sh.tok[i * K + lane] = ti;
            if (topk_token) topk_token[row * K + lane] = ti;
            if (topk_logprob) topk_logprob[row * K + lane] = lq;
        }
    }
    if (tid < kMaxL + 2) { sh.lvl_cnt[tid] = 0; sh.lvl_cur[tid] = 0; }
    __syncthreads();

    // ---- 2. best-first selection (Algorithm 1) on warp 0 ---------------------------------------
    if (warp == 0) {
        int count = 1;
        if (lane == 0) {
            sh.sigma[0] = 0.f; sh.depth[0] = 0; sh.cc[0] = 0; sh.parent[0] = -1; sh.rank[0] = 0;
            sh.cand[0] = sh.logq[0];
        }
        float bestv = lane == 0 ? sh.logq[0] : -CUDART_INF_F;
        int bests = lane == 0 ? 0 : -1;
        const unsigned none = orderable(-CUDART_INF_F);
        __syncwarp();
        for (int t = 0; t < B; ++t) {
            const unsigned key = orderable(bestv);
            const unsigned mx = __reduce_max_sync(kFull, key);
            if (mx == none) break;  // heap empty: fewer than B prefixes exist in S_K
            const int src = __ffs(__ballot_sync(kFull, key == mx)) - 1;
            const int u = __shfl_sync(kFull, bests, src);
            const float v = from_orderable(mx);  // the winning candidate's score
            const int du = sh.depth[u], cu = sh.cc[u];
            const float su = sh.sigma[u];
            const int n = count++;
            // This lane's best among its slots other than u (slot s sits on lane s % 32; n is not written
            // yet).  These reads depend on nothing the pop computes, so they travel with the reads of
            // u's state; the two slots that change are patched in from registers below.  The trip count
            // is the same for every lane: a loop that lanes leave at different times costs the warp
            // about 150 cycles per pop.
            bestv = -CUDART_INF_F; bests = -1;
            auto look = [&](int i) {
                const int j = i * 32 + lane;
                const float cj = sh.cand[min(j, n - 1)];
                const float c = ((j < n) & (j != u)) ? cj : -CUDART_INF_F;
                const bool up = c > bestv;
                bestv = up ? c : bestv;
                bests = up ? j : bests;
            };
            if (B < 128) {  // at most 4 slots per lane: straight-line code, the reads leave together
#pragma unroll
                for (int i = 0; i < 4; ++i) look(i);
            } else {
                const int trips = (n + 31) >> 5;
#pragma unroll 4
                for (int i = 0; i < trips; ++i) look(i);
            }
            const float cand_u = (cu + 1 < K) ? su + sh.logq[du * K + cu + 1] : -CUDART_INF_F;
            const float cand_n = (du + 1 < L) ? v + sh.logq[(du + 1) * K] : -CUDART_INF_F;
            // within a lane equal scores go to the lower slot; across lanes the pop takes the lowest lane (any
            // order of equal scores is a valid pop order: the contract is the node set)
            const bool take_u = (lane == (u & 31)) & ((cand_u > bestv) | ((cand_u == bestv) & (u < bests)));
            bestv = take_u ? cand_u : bestv;
            bests = take_u ? u : bests;
            const bool take_n = (lane == (n & 31)) & (cand_n > bestv);
            bestv = take_n ? cand_n : bestv;
            bests = take_n ? n : bests;
            __syncwarp();  // all lanes have read u's state and their slots before lane 0 overwrites them
            {   // lane 0 writes; the other lanes store the same values to a spare slot instead of branching
                const int wn = lane == 0 ? n : kSlots - 1, wu = lane == 0 ? u : kSlots - 1;
                sh.parent[wn] = static_cast<short>(u);
                sh.rank[wn] = static_cast<unsigned char>(cu + 1);
                sh.depth[wn] = static_cast<unsigned char>(du + 1);
                sh.sigma[wn] = v;
                sh.cc[wn] = 0;
                sh.cand[wn] = cand_n;
                sh.cc[wu] = static_cast<unsigned char>(cu + 1);
                sh.cand[wu] = cand_u;
            }
            __syncwarp();
        }
        __syncwarp();

        // ---- 3. level order: rows sorted by (depth, parent row, rank) --------------------------
        for (int j = lane; j < count; j += 32) atomicAdd(&sh.lvl_cnt[sh.depth[j]], 1);
        __syncwarp();
        if (lane == 0) {
            int acc = 0;
            for (int d = 0; d <= L + 1; ++d) { sh.lvl_start[d] = acc; if (d <= L) acc += sh.lvl_cnt[d]; }
            sh.lvl_start[L + 2] = acc;
            sh.row_of[0] = 0; sh.inv[0] = 0;
            sh.count = count;
        }
        __syncwarp();
        for (int j = lane; j < count; j += 32) {
            const int d = sh.depth[j];
            sh.bucket[sh.lvl_start[d] + atomicAdd(&sh.lvl_cur[d], 1)] = static_cast<short>(j);
        }
        __syncwarp();
        for (int d = 0; d <= L; ++d) {
            const int lo = sh.lvl_start[d], hi = sh.lvl_start[d + 1], next = hi;
            if (lo == hi) break;
            int carry = 0;
            for (int base = lo; base < hi; base += 32) {
                const int row = base + lane;
                const bool ok = row < hi;
                const int c = ok ? sh.cc[sh.inv[row]] : 0;
                int incl = c;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int t = __shfl_up_sync(kFull, incl, o);
                    if (lane >= o) incl += t;
                }
                if (ok) sh.fc[row] = static_cast<short>(c ? next + carry + incl - c : -1);
                carry += __shfl_sync(kFull, incl, 31);
            }
            __syncwarp();
            if (d < L) {
                for (int idx = sh.lvl_start[d + 1] + lane; idx < sh.lvl_start[d + 2]; idx += 32) {
                    const int n = sh.bucket[idx];
                    const int row = sh.fc[sh.row_of[sh.parent[n]]] + sh.rank[n] - 1;
                    sh.row_of[n] = static_cast<short>(row);
                    sh.inv[row] = static_cast<short>(n);
                }
            }
            __syncwarp();
        }
    }
    __syncthreads();

    // ---- 4. write the verifier's inputs --------------------------------------------------------
    const int count = sh.count;
    const size_t o = static_cast<size_t>(r) * N;
    const int P = prefix_len[r];
    if (tid == 0) n_rows[r] = count;
    for (int row = tid; row < N; row += kThreads) {
        int tokv = -1, par = -1, dep = -1, pos = -1, fcv = -1, ccv = 0;
        float lp = 0.f;
        if (row < count) {
            const int s = sh.inv[row];
            dep = sh.depth[s];
            tokv = row == 0 ? root_token[r] : sh.tok[(dep - 1) * K + sh.rank[s] - 1];
            par = row == 0 ? -1 : sh.row_of[sh.parent[s]];
            pos = P + dep;
            fcv = sh.fc[row];
            ccv = sh.cc[s];
            lp = sh.sigma[s];
        }
        sh.prow[row] = static_cast<short>(par);
        node_token[o + row] = tokv;
        node_parent[o + row] = par;
        node_depth[o + row] = dep;
        position_ids[o + row] = pos;
        if (first_child) first_child[o + row] = fcv;
        if (child_count) child_count[o + row] = ccv;
        if (node_logprob) node_logprob[o + row] = lp;
    }
    __syncthreads();
    // ancestor-or-self bits: walk up the parent chain (rows strictly decrease towards the root)
    for (int idx = tid; idx < N * W; idx += kThreads) {
        const int row = idx / W, w = idx % W;
        uint32_t bits = 0;
        if (row < count) {
            int a = row;
            while (a >= w * 32) {
                if (a < (w + 1) * 32) bits |= 1u << (a & 31);
                a = sh.prow[a];
            }
        }
        anc_mask[o * W + idx] = bits;
    }
}

}  // namespace

cudaError_t launch_tree_build(int R, int L, int V, int K, int B, const BuildPartialLayout& lay, const void* ws,
                              const void* logits, int dt, int64_t row_stride,
                              const int32_t* root_token, const int32_t* prefix_len,
                              int32_t* n_rows, int32_t* node_token, int32_t* node_parent, int32_t* node_depth,
                              int32_t* position_ids, uint32_t* anc_mask, int32_t* first_child,
                              int32_t* child_count, float* node_logprob, int32_t* topk_token,
                              float* topk_logprob, cudaStream_t st) {
    const char* w = static_cast<const char*>(ws);
    const float* pm = reinterpret_cast<const float*>(w + lay.off_m);
    const float* ps = reinterpret_cast<const float*>(w + lay.off_s);
    const float* tmax = reinterpret_cast<const float*>(w + lay.off_tmax);
    const float* wmax = reinterpret_cast<const float*>(w + lay.off_wmax);
    if (dt == DDTREE_F32)
        return launch_pdl(tree_build_kernel<float>, dim3(R), dim3(kThreads), 0, st,
            L, V, K, B, lay.chunks, pm, ps, tmax, wmax, static_cast<const float*>(logits), row_stride, root_token, prefix_len,
            n_rows, node_token, node_parent, node_depth, position_ids, anc_mask, first_child, child_count, node_logprob,
            topk_token, topk_logprob);
    return launch_pdl(tree_build_kernel<__nv_bfloat16>, dim3(R), dim3(kThreads), 0, st,
            L, V, K, B, lay.chunks, pm, ps, tmax, wmax, static_cast<const __nv_bfloat16*>(logits), row_stride, root_token,
            prefix_len, n_rows, node_token, node_parent, node_depth, position_ids, anc_mask, first_child, child_count,
            node_logprob, topk_token, topk_logprob);
}

}  // namespace ddtree

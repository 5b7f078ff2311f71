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

__device__ __forceinline__ unsigned orderable(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
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
    int lvl_cnt[kMaxL + 2];
    int lvl_start[kMaxL + 3];
    int lvl_cur[kMaxL + 2];
    int count;
};

__global__ void __launch_bounds__(kThreads)
tree_build_kernel(int L, int K, int B, int chunks, const float* __restrict__ pm, const float* __restrict__ ps,
                  const float* __restrict__ pval, const int* __restrict__ pid,
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

        // K best of chunks*K candidates, (value desc, id asc); lane k ends up with rank k+1
        float tv = -CUDART_INF_F, thr_v = -CUDART_INF_F;
        int ti = -1, thr_i = -1;
        const int total = chunks * K;
        const float* cv = pval + row * total;
        const int* ci = pid + row * total;
        for (int j0 = 0; j0 < total; j0 += 32) {
            const int j = j0 + lane;
            const float v = j < total ? cv[j] : -CUDART_INF_F;
            const int id = j < total ? ci[j] : -1;
            unsigned any = __ballot_sync(kFull, beats(v, id, thr_v, thr_i));
            while (any) {
                const int src = __ffs(any) - 1;
                any &= any - 1;
                const float sv = __shfl_sync(kFull, v, src);
                const int si = __shfl_sync(kFull, id, src);
                if (beats(sv, si, thr_v, thr_i)) {
                    const int pos = __popc(__ballot_sync(kFull, beats(tv, ti, sv, si)));
                    const float upv = __shfl_up_sync(kFull, tv, 1);
                    const int upi = __shfl_up_sync(kFull, ti, 1);
                    if (lane == pos) { tv = sv; ti = si; }
                    else if (lane > pos) { tv = upv; ti = upi; }
                    thr_v = __shfl_sync(kFull, tv, K - 1);
                    thr_i = __shfl_sync(kFull, ti, K - 1);
                }
            }
        }
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
            const float v = __shfl_sync(kFull, bestv, src);
            const int du = sh.depth[u], cu = sh.cc[u];
            const float su = sh.sigma[u];
            const int n = count++;
            const float cand_u = (cu + 1 < K) ? su + sh.logq[du * K + cu + 1] : -CUDART_INF_F;
            const float cand_n = (du + 1 < L) ? v + sh.logq[(du + 1) * K] : -CUDART_INF_F;
            __syncwarp();  // all lanes have read u's state before lane 0 overwrites it
            if (lane == 0) {
                sh.parent[n] = static_cast<short>(u);
                sh.rank[n] = static_cast<unsigned char>(cu + 1);
                sh.depth[n] = static_cast<unsigned char>(du + 1);
                sh.sigma[n] = v;
                sh.cc[n] = 0;
                sh.cc[u] = static_cast<unsigned char>(cu + 1);
                sh.cand[u] = cand_u;
                sh.cand[n] = cand_n;
            }
            __syncwarp();
            if (lane == (u & 31)) {  // this lane's best was consumed: rescan its slots
                bestv = -CUDART_INF_F; bests = -1;
                for (int j = lane; j < count; j += 32) {
                    const float c = sh.cand[j];
                    if (c > bestv) { bestv = c; bests = j; }
                }
            } else if (lane == (n & 31)) {
                if (cand_n > bestv) { bestv = cand_n; bests = n; }
            }
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

cudaError_t launch_tree_build(int R, int L, int K, int B, const BuildPartialLayout& lay, const void* ws,
                              const int32_t* root_token, const int32_t* prefix_len,
                              int32_t* n_rows, int32_t* node_token, int32_t* node_parent, int32_t* node_depth,
                              int32_t* position_ids, uint32_t* anc_mask, int32_t* first_child,
                              int32_t* child_count, float* node_logprob, int32_t* topk_token,
                              float* topk_logprob, cudaStream_t st) {
    const char* w = static_cast<const char*>(ws);
    tree_build_kernel<<<R, kThreads, 0, st>>>(
        L, K, B, lay.chunks, reinterpret_cast<const float*>(w + lay.off_m),
        reinterpret_cast<const float*>(w + lay.off_s), reinterpret_cast<const float*>(w + lay.off_val),
        reinterpret_cast<const int*>(w + lay.off_id), root_token, prefix_len, n_rows, node_token, node_parent,
        node_depth, position_ids, anc_mask, first_child, child_count, node_logprob, topk_token, topk_logprob);
    return cudaGetLastError();
}

}  // namespace ddtree

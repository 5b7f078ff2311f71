// One CTA per request: reduce the per-chunk (max, argmax) partials of the target logits to the
// target's greedy choice at every row (or take the choices drawn by the sampling pass), then walk the tree from the root, following the child whose
// token equals that choice until none matches (Section 4.4, Figure 2(b)).
#include "common.cuh"
#include <math_constants.h>

namespace ddtree {
namespace {

constexpr int kThreads = 256;
constexpr unsigned kFull = 0xffffffffu;

__global__ void __launch_bounds__(kThreads)
accept_walk_kernel(int N, int L, int chunks, const float* __restrict__ pval, const int* __restrict__ pid,
                   const int32_t* __restrict__ choice, const int32_t* __restrict__ node_token, const int32_t* __restrict__ node_parent,
                   const int32_t* __restrict__ n_rows, int32_t* __restrict__ accept_len,
                   int32_t* __restrict__ accept_nodes, int32_t* __restrict__ accept_tokens,
                   int32_t* __restrict__ bonus_token, int32_t* __restrict__ node_argmax) {
    __shared__ int s_choice[kMaxN];
    __shared__ int s_token[kMaxN];
    __shared__ short s_parent[kMaxN];
    const int r = blockIdx.x, tid = threadIdx.x;
    pdl_wait();
    const int n = min(n_rows[r], N);
    const size_t o = static_cast<size_t>(r) * N;
    for (int row = tid; row < N; row += kThreads) {
        int best = -1;
        if (row < n) {
            if (choice) {  // the target's choice was drawn by the sampling pass
                best = choice[o + row];
            } else {
                const float* v = pval + (o + row) * chunks;
                const int* id = pid + (o + row) * chunks;
                float bv = v[0];
                best = id[0];
                for (int c = 1; c < chunks; ++c)
                    if (beats(v[c], id[c], bv, best)) { bv = v[c]; best = id[c]; }
            }
            s_token[row] = node_token[o + row];
            s_parent[row] = static_cast<short>(node_parent[o + row]);
        }
        s_choice[row] = best;
        if (node_argmax) node_argmax[o + row] = best;
    }
    __syncthreads();
    if (tid >= 32) return;
    const int lane = tid;
    int cur = 0, len = 0;
    while (len < L) {
        const int want = s_choice[cur];
        int found = -1;
        for (int base = cur + 1; base < n && found < 0; base += 32) {  // children have larger rows
            const int j = base + lane;
            const bool hit = j < n && s_parent[j] == cur && s_token[j] == want;
            const unsigned m = __ballot_sync(kFull, hit);
            if (m) found = base + __ffs(m) - 1;
        }
        if (found < 0) break;
        if (lane == 0) {
            accept_nodes[static_cast<size_t>(r) * L + len] = found;
            accept_tokens[static_cast<size_t>(r) * L + len] = s_token[found];
        }
        cur = found;
        ++len;
    }
    for (int k = len + lane; k < L; k += 32) {
        accept_nodes[static_cast<size_t>(r) * L + k] = -1;
        accept_tokens[static_cast<size_t>(r) * L + k] = -1;
    }
    if (lane == 0) {
        accept_len[r] = len;
        bonus_token[r] = s_choice[cur];
    }
}

}  // namespace

cudaError_t launch_accept_walk(int R, int N, int L, const ArgmaxLayout& lay, const void* ws, const int32_t* choice,
                               const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows,
                               int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                               int32_t* bonus_token, int32_t* node_argmax, cudaStream_t st) {
    const char* w = static_cast<const char*>(ws);
    return launch_pdl(accept_walk_kernel, dim3(R), dim3(kThreads), 0, st, N, L, lay.chunks,
                      reinterpret_cast<const float*>(w + lay.off_val), reinterpret_cast<const int*>(w + lay.off_id), choice,
                      node_token, node_parent, n_rows, accept_len, accept_nodes, accept_tokens, bonus_token, node_argmax);
}

}  // namespace ddtree

// End of a round (Section 4.4): only the accepted path stays in the KV cache.  For every layer and
// request the key and value rows of the root and of the accepted nodes are copied from this
// round's tree buffers to consecutive cache rows, root first, so that the i-th accepted node lands
// at the position id it was verified at.  Pure data movement: one CTA per (layer, request, path
// position) moves one K row and one V row with 16-byte accesses; all layers go in one launch.
#include "common.cuh"

namespace ddtree {

namespace {

struct CompactParams {
    const void* k_tree[kCompactLayersPerLaunch];
    const void* v_tree[kCompactLayersPerLaunch];
    void* k_cache[kCompactLayersPerLaunch];
    void* v_cache[kCompactLayersPerLaunch];
    const int64_t* dst_row;
    const int32_t* accept_len;
    const int32_t* accept_nodes;
    int N, L;
    int row_vec16;  // 16-byte vectors per row (Hkv * d * element size / 16)
};

__global__ void __launch_bounds__(128)
kv_compact_kernel(const CompactParams p) {
    pdl_wait();
    const int i = blockIdx.x;          // 0 = root, 1.. = accepted nodes in path order
    const int r = blockIdx.y, layer = blockIdx.z;
    const int a = min(max(p.accept_len[r], 0), p.L);
    if (i > a) return;
    const int node = i == 0 ? 0 : p.accept_nodes[static_cast<size_t>(r) * p.L + i - 1];
    if (node < 0 || node >= p.N) return;  // never true for the outputs of ddtree_accept
    const size_t src = (static_cast<size_t>(r) * p.N + node) * p.row_vec16;
    const size_t dst = static_cast<size_t>(p.dst_row[r] + i) * p.row_vec16;
    const uint4* ks = static_cast<const uint4*>(p.k_tree[layer]) + src;
    const uint4* vs = static_cast<const uint4*>(p.v_tree[layer]) + src;
    uint4* kd = static_cast<uint4*>(p.k_cache[layer]) + dst;
    uint4* vd = static_cast<uint4*>(p.v_cache[layer]) + dst;
    for (int c = threadIdx.x; c < p.row_vec16; c += blockDim.x) {
        kd[c] = ks[c];
        vd[c] = vs[c];
    }
}

}  // namespace

cudaError_t launch_kv_compact(int R, int N, int L, int row_bytes, int layers, const void* const* k_tree,
                              const void* const* v_tree, void* const* k_cache, void* const* v_cache,
                              const int64_t* dst_row, const int32_t* accept_len, const int32_t* accept_nodes,
                              cudaStream_t st) {
    for (int l0 = 0; l0 < layers; l0 += kCompactLayersPerLaunch) {
        const int nl = layers - l0 < kCompactLayersPerLaunch ? layers - l0 : kCompactLayersPerLaunch;
        CompactParams p;
        for (int l = 0; l < nl; ++l) {
            p.k_tree[l] = k_tree[l0 + l]; p.v_tree[l] = v_tree[l0 + l];
            p.k_cache[l] = k_cache[l0 + l]; p.v_cache[l] = v_cache[l0 + l];
        }
        for (int l = nl; l < kCompactLayersPerLaunch; ++l) { p.k_tree[l] = p.v_tree[l] = nullptr; p.k_cache[l] = p.v_cache[l] = nullptr; }
        p.dst_row = dst_row; p.accept_len = accept_len; p.accept_nodes = accept_nodes;
        p.N = N; p.L = L; p.row_vec16 = row_bytes / 16;
        const cudaError_t e = launch_pdl(kv_compact_kernel, dim3(L + 1, R, nl), dim3(128), 0, st, p);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

}  // namespace ddtree

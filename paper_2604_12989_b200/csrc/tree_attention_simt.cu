// Tree attention with plain FMA arithmetic (fp32 accumulate), one warp per (request, row, head).
// Implements Section 4.4's rule directly: row i attends to every cached key of its request and to
// the tree rows whose bit is set in its ancestor mask.  This is the path for fp32 tensors, where
// the 1e-4 tolerance rules out reduced-precision tensor-core inputs; it is not tuned for speed.
#include "common.cuh"
#include <math_constants.h>

namespace ddtree {
namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr int kWarpsPerCta = 4;
constexpr float kLog2e = 1.4426950408889634f;

template <int D>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
tree_attention_f32_kernel(const float* __restrict__ q, const float* __restrict__ k_cache,
                          const float* __restrict__ v_cache, const float* __restrict__ k_tree,
                          const float* __restrict__ v_tree, const int32_t* __restrict__ cu_prefix,
                          const uint32_t* __restrict__ anc_mask, const int32_t* __restrict__ n_rows,
                          float* __restrict__ out, float* __restrict__ lse, int R, int N, int W, int Hq, int Hkv,
                          float scale_log2) {
    constexpr int E = D / 32;  // output elements per lane
    __shared__ float s_q[kWarpsPerCta][D];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    pdl_wait();  // n_rows and the mask may come from the kernel launched just before
    const long long task = static_cast<long long>(blockIdx.x) * kWarpsPerCta + warp;
    if (task >= static_cast<long long>(R) * N * Hq) return;
    const int h = static_cast<int>(task % Hq);
    const int i = static_cast<int>((task / Hq) % N);
    const int r = static_cast<int>(task / (static_cast<long long>(Hq) * N));
    const int n = n_rows[r];
    if (i >= n) return;
    const int kv = h / (Hq / Hkv);
    const int p0 = cu_prefix[r], P = cu_prefix[r + 1] - p0;

    const float* qrow = q + ((static_cast<size_t>(r) * N + i) * Hq + h) * D;
    for (int e = lane; e < D; e += 32) s_q[warp][e] = qrow[e] * scale_log2;
    __syncwarp();

    float m = -CUDART_INF_F, l = 0.f;
    float acc[E];
#pragma unroll
    for (int e = 0; e < E; ++e) acc[e] = 0.f;

    const uint32_t* mrow = anc_mask + (static_cast<size_t>(r) * N + i) * W;
    const int prefix_tiles = (P + 31) / 32, tree_tiles = (n + 31) / 32;
    for (int t = 0; t < prefix_tiles + tree_tiles; ++t) {
        const bool in_prefix = t < prefix_tiles;
        const int j = (in_prefix ? t : t - prefix_tiles) * 32 + lane;
        bool vis;
        const float *krow, *vbase;
        if (in_prefix) {
            vis = j < P;
            krow = k_cache + ((static_cast<size_t>(p0) + j) * Hkv + kv) * D;
            vbase = v_cache + ((static_cast<size_t>(p0) + (t * 32)) * Hkv + kv) * D;
        } else {
            vis = j < n && ((mrow[t - prefix_tiles] >> lane) & 1u);
            krow = k_tree + ((static_cast<size_t>(r) * N + j) * Hkv + kv) * D;
            vbase = v_tree + ((static_cast<size_t>(r) * N + (t - prefix_tiles) * 32) * Hkv + kv) * D;
        }
        const unsigned any = __ballot_sync(kFull, vis);
        if (!any) continue;
        float s = -CUDART_INF_F;
        if (vis) {
            float dot = 0.f;
#pragma unroll 8
            for (int e = 0; e < D; e += 4) {
                const float4 kk = __ldg(reinterpret_cast<const float4*>(krow + e));
                dot = fmaf(kk.x, s_q[warp][e], dot);
                dot = fmaf(kk.y, s_q[warp][e + 1], dot);
                dot = fmaf(kk.z, s_q[warp][e + 2], dot);
                dot = fmaf(kk.w, s_q[warp][e + 3], dot);
            }
            s = dot;  // already in log2 units (q was pre-multiplied by scale*log2(e))
        }
        float tm = s;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) tm = fmaxf(tm, __shfl_xor_sync(kFull, tm, o));
        const float m_new = fmaxf(m, tm);
        const float alpha = exp2f(m - m_new);  // m = -inf on the first visible tile: alpha = 0
        const float p = vis ? exp2f(s - m_new) : 0.f;
        float ps = p;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) ps += __shfl_xor_sync(kFull, ps, o);
        l = l * alpha + ps;
        m = m_new;
#pragma unroll
        for (int e = 0; e < E; ++e) acc[e] *= alpha;
        // value rows of the visible keys, eight at a time: their loads leave together (a row that is not visible is
        // not read at all: it may lie outside the request, or hold anything)
        for (int s0 = 0; s0 < 32; s0 += 8) {
            if (!((any >> s0) & 0xffu)) continue;  // warp-uniform
            float pj[8], vv[8][E];
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const bool on = (any >> (s0 + u)) & 1u;
                pj[u] = __shfl_sync(kFull, p, s0 + u);
                const float* vrow = vbase + static_cast<size_t>(s0 + u) * Hkv * D;
#pragma unroll
                for (int e = 0; e < E; ++e) vv[u][e] = on ? __ldg(vrow + e * 32 + lane) : 0.f;
            }
#pragma unroll
            for (int u = 0; u < 8; ++u)
#pragma unroll
                for (int e = 0; e < E; ++e) acc[e] = fmaf(pj[u], vv[u][e], acc[e]);
        }
    }
    float* orow = out + ((static_cast<size_t>(r) * N + i) * Hq + h) * D;
    const float inv = 1.f / l;
#pragma unroll
    for (int e = 0; e < E; ++e) orow[e * 32 + lane] = acc[e] * inv;
    if (lse && lane == 0) lse[(static_cast<size_t>(r) * N + i) * Hq + h] = (m + log2f(l)) / kLog2e;
}

}  // namespace

cudaError_t launch_tree_attention_f32(const AttnArgs& a, cudaStream_t st) {
    const long long tasks = static_cast<long long>(a.R) * a.N * a.Hq;
    const unsigned grid = static_cast<unsigned>((tasks + kWarpsPerCta - 1) / kWarpsPerCta);
    const float scale_log2 = a.scale * kLog2e;
    const float* q = static_cast<const float*>(a.q);
    const float* kc = static_cast<const float*>(a.k_cache);
    const float* vc = static_cast<const float*>(a.v_cache);
    const float* kt = static_cast<const float*>(a.k_tree);
    const float* vt = static_cast<const float*>(a.v_tree);
    float* out = static_cast<float*>(a.out);
    if (a.d == 64)
        return launch_pdl(tree_attention_f32_kernel<64>, dim3(grid), dim3(kWarpsPerCta * 32), 0, st, q, kc, vc, kt, vt,
                          a.cu_prefix, a.anc_mask, a.n_rows, out, a.lse, a.R, a.N, a.W, a.Hq, a.Hkv, scale_log2);
    return launch_pdl(tree_attention_f32_kernel<128>, dim3(grid), dim3(kWarpsPerCta * 32), 0, st, q, kc, vc, kt, vt,
                      a.cu_prefix, a.anc_mask, a.n_rows, out, a.lse, a.R, a.N, a.W, a.Hq, a.Hkv, scale_log2);
}

}  // namespace ddtree

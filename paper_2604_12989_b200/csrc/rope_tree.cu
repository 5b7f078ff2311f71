// Rotary positional encoding of the tree's query and key rows at the position ids ddtree_build assigned
// (Section 4.4: position ids follow the tree depth, so that every node is encoded at the position it would have
// in its own branch).
// Pair (j, j + d/2) of every head of row i is rotated by position_ids[i] * theta^(-2j/d) (half-split form).
//
// A pass of its own, in place, before the attention call rather than a step of the attention kernel's load
// path: a tree K row is loaded by every row tile, KV split and query-head group that attends to it, and a Q
// tile by every KV split, so rotating at load time would redo the same rotation in each of those CTAs.  One
// CTA per tree row: the d/2 angles of the row are formed and reduced modulo 2 pi in double precision (positions
// reach 10^5, where a float32 angle is off by 10^-2 rad; the frequencies theta^(-2j/d) come from the host as
// doubles), their sine and cosine are taken in float32 on the reduced angle, and the rotation is applied to all
// query and KV heads of the row.
#include "common.cuh"
#include <cmath>

namespace ddtree {
namespace {

constexpr int kThreads = 128;
constexpr int kMaxHalf = 128;  // head_dim <= 256

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_f32(float* p, float v) { *p = v; }
__device__ __forceinline__ void from_f32(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

struct RopeFreq {
    double inv_freq[kMaxHalf];  // theta^(-2j/d)
};

template <typename T>
__global__ void __launch_bounds__(kThreads)
rope_tree_kernel(T* __restrict__ q, T* __restrict__ k, const int32_t* __restrict__ position_ids,
                 const int32_t* __restrict__ n_rows, int N, int Hq, int Hkv, int d, int vectors,
                 const __grid_constant__ RopeFreq f) {
    __shared__ float cs[2][kMaxHalf];
    pdl_wait();
    const int row = blockIdx.x, tid = threadIdx.x;
    if (row % N >= n_rows[row / N]) return;  // padding rows are left alone
    const int half = d / 2;
    const double pos = static_cast<double>(position_ids[row]);
    for (int j = tid; j < half; j += kThreads) {
        // angle modulo 2 pi in double (2 pi split into a leading part and its remainder), then float32 sincos on
        // an argument in [-pi, pi]: a handful of double operations instead of a double-precision sincos
        const double a = pos * f.inv_freq[j];
        const double turns = rint(a * 0.15915494309189535);
        const double red = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, a));
        float s, c;
        sincosf(static_cast<float>(red), &s, &c);
        cs[0][j] = c;
        cs[1][j] = s;
    }
    __syncthreads();
    const int q_heads = q ? Hq : 0, heads = q_heads + (k ? Hkv : 0);
    constexpr int VN = 16 / sizeof(T);  // elements per 16-byte access
    if (vectors) {  // half is a multiple of VN and the tensors are 16-byte aligned: 16-byte accesses
        const int per_head = half / VN;
        for (int idx = tid; idx < heads * per_head; idx += kThreads) {
            const int h = idx / per_head, j = (idx - h * per_head) * VN;
            T* p = h < q_heads ? q + (static_cast<size_t>(row) * Hq + h) * d
                               : k + (static_cast<size_t>(row) * Hkv + (h - q_heads)) * d;
            uint4 xv = *reinterpret_cast<const uint4*>(p + j), yv = *reinterpret_cast<const uint4*>(p + j + half);
            T* xe = reinterpret_cast<T*>(&xv);
            T* ye = reinterpret_cast<T*>(&yv);
#pragma unroll
            for (int e = 0; e < VN; ++e) {
                const float x = to_f32(xe[e]), y = to_f32(ye[e]);
                const float c = cs[0][j + e], s = cs[1][j + e];
                from_f32(xe + e, x * c - y * s);
                from_f32(ye + e, y * c + x * s);
            }
            *reinterpret_cast<uint4*>(p + j) = xv;
            *reinterpret_cast<uint4*>(p + j + half) = yv;
        }
        return;
    }
    for (int idx = tid; idx < heads * half; idx += kThreads) {
        const int h = idx / half, j = idx - h * half;
        T* p = h < q_heads ? q + (static_cast<size_t>(row) * Hq + h) * d
                           : k + (static_cast<size_t>(row) * Hkv + (h - q_heads)) * d;
        const float x = to_f32(p[j]), y = to_f32(p[j + half]);
        const float c = cs[0][j], s = cs[1][j];
        from_f32(p + j, x * c - y * s);
        from_f32(p + j + half, y * c + x * s);
    }
}

}  // namespace

cudaError_t launch_rope_tree(void* q, void* k, const int32_t* position_ids, const int32_t* n_rows, int dt, int R, int N,
                             int Hq, int Hkv, int d, double log2_theta, cudaStream_t st) {
    const dim3 grid(static_cast<unsigned>(R) * N);
    RopeFreq f;
    for (int j = 0; j < kMaxHalf; ++j) f.inv_freq[j] = j < d / 2 ? std::exp2(-(2.0 * j / d) * log2_theta) : 0.0;
    const int vn = dt == DDTREE_F32 ? 4 : 8;
    const int vectors = ((d / 2) % vn == 0 && (reinterpret_cast<uintptr_t>(q) & 15u) == 0 &&
                         (reinterpret_cast<uintptr_t>(k) & 15u) == 0) ? 1 : 0;
    if (dt == DDTREE_F32)
        return launch_pdl(rope_tree_kernel<float>, grid, dim3(kThreads), 0, st, static_cast<float*>(q), static_cast<float*>(k),
                          position_ids, n_rows, N, Hq, Hkv, d, vectors, f);
    return launch_pdl(rope_tree_kernel<__nv_bfloat16>, grid, dim3(kThreads), 0, st, static_cast<__nv_bfloat16*>(q),
                      static_cast<__nv_bfloat16*>(k), position_ids, n_rows, N, Hq, Hkv, d, vectors, f);
}

}  // namespace ddtree

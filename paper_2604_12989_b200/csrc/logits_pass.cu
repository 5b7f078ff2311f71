// Vocabulary-wide passes over logits rows (HBM-bound):
//   logits_topk_kernel  -- per (row, chunk): running max, sum of exponentials and the K best
//                          (value, id) pairs of the chunk (Sections 3 and 4.3: q_i = softmax(l_i),
//                          tokens ranked by probability).
//   row_argmax_kernel   -- per (row, chunk): maximum and the lowest id attaining it (the greedy
//                          decoding rule of Section 4.4).
// Both read each element once with 16-byte loads; chunk partials are merged by the kernels in
// tree_build.cu / accept_walk.cu.
#include "common.cuh"
#include <math_constants.h>

namespace ddtree {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kUnroll = 4;
constexpr float kLog2e = 1.4426950408889634f;
constexpr unsigned kFull = 0xffffffffu;

template <typename T> struct Vec16;
template <> struct Vec16<float> {
    static constexpr int N = 4;
    static __device__ __forceinline__ void load(const float* p, float (&v)[4]) {
        float4 t = __ldg(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    static __device__ __forceinline__ float scalar(const float* p) { return __ldg(p); }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&v)[8]) {
        uint4 t = __ldg(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ float scalar(const __nv_bfloat16* p) {
        return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
};

// Sorted list of the best entries seen by a warp: lane k holds the k-th best (value, id).
struct WarpTopK {
    float tv;   // this lane's entry
    int ti;
    float thr_v;  // entry of lane K-1 (what a candidate has to beat)
    int thr_i;
    __device__ __forceinline__ void init() { tv = -CUDART_INF_F; ti = -1; thr_v = -CUDART_INF_F; thr_i = -1; }
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

__device__ __forceinline__ void online_merge(float& m, float& s, float m2, float s2) {
    const float M = fmaxf(m, m2);
    if (M == -CUDART_INF_F) { m = M; s = 0.f; return; }
    s = s * exp2f((m - M) * kLog2e) + s2 * exp2f((m2 - M) * kLog2e);
    m = M;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
logits_topk_kernel(const T* __restrict__ logits, int64_t row_stride, int V, int K, int chunk_elems, int chunks,
                   float* __restrict__ pm, float* __restrict__ ps, float* __restrict__ pval,
                   int* __restrict__ pid) {
    constexpr int VN = Vec16<T>::N;
    const int row = blockIdx.x / chunks, chunk = blockIdx.x % chunks;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* x = logits + static_cast<int64_t>(row) * row_stride;
    const int begin = chunk * chunk_elems;
    const int end = min(V, begin + chunk_elems);
    const int vec_end = begin + ((end - begin) / VN) * VN;

    WarpTopK top;
    top.init();
    float m = -CUDART_INF_F, s = 0.f;

    constexpr int kStep = kThreads * VN;
    for (int it = begin + warp * 32 * VN; it < vec_end; it += kUnroll * kStep) {
        float vals[kUnroll][VN];
        int id0[kUnroll];
        bool ok[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            id0[u] = it + u * kStep + lane * VN;
            ok[u] = id0[u] < vec_end;
            if (ok[u]) Vec16<T>::load(x + id0[u], vals[u]);
            else {
#pragma unroll
                for (int e = 0; e < VN; ++e) vals[u][e] = -CUDART_INF_F;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (it + u * kStep >= vec_end) break;  // warp-uniform
            if (ok[u]) {
                float vm = vals[u][0];
#pragma unroll
                for (int e = 1; e < VN; ++e) vm = fmaxf(vm, vals[u][e]);
                if (vm > m) { s *= exp2f((m - vm) * kLog2e); m = vm; }
#pragma unroll
                for (int e = 0; e < VN; ++e) s += exp2f((vals[u][e] - m) * kLog2e);
            }
            top.offer<VN>(vals[u], id0[u], K, lane);
        }
    }
    // ragged tail of the row (fewer than VN elements), one element per lane of warp 0
    if (warp == 0 && vec_end < end) {
        float v1[1];
        const int id = vec_end + lane;
        const bool ok = id < end;
        v1[0] = ok ? Vec16<T>::scalar(x + id) : -CUDART_INF_F;
        if (ok) {
            if (v1[0] > m) { s *= exp2f((m - v1[0]) * kLog2e); m = v1[0]; }
            s += exp2f((v1[0] - m) * kLog2e);
        }
        top.offer<1>(v1, id, K, lane);
    }

    // block-level merge
    __shared__ float sm_v[kWarps][32];
    __shared__ int sm_i[kWarps][32];
    __shared__ float sm_m[kWarps], sm_s[kWarps];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(kFull, m, o);
        const float s2 = __shfl_xor_sync(kFull, s, o);
        online_merge(m, s, m2, s2);
    }
    sm_v[warp][lane] = lane < K ? top.tv : -CUDART_INF_F;
    sm_i[warp][lane] = lane < K ? top.ti : -1;
    if (lane == 0) { sm_m[warp] = m; sm_s[warp] = s; }
    __syncthreads();
    if (warp == 0) {
        for (int w = 1; w < kWarps; ++w) {
            float v1[1] = {sm_v[w][lane]};
            // ids are absolute, so offer() is called with a per-lane id and a single element
            const int id = sm_i[w][lane];
            unsigned any = __ballot_sync(kFull, beats(v1[0], id, top.thr_v, top.thr_i));
            while (any) {
                const int src = __ffs(any) - 1;
                any &= any - 1;
                const float v = __shfl_sync(kFull, v1[0], src);
                const int vi = __shfl_sync(kFull, id, src);
                if (beats(v, vi, top.thr_v, top.thr_i)) top.insert(v, vi, K, lane);
            }
            online_merge(m, s, sm_m[w], sm_s[w]);
        }
        const size_t p = static_cast<size_t>(row) * chunks + chunk;
        if (lane < K) { pval[p * K + lane] = top.tv; pid[p * K + lane] = top.ti; }
        if (lane == 0) { pm[p] = m; ps[p] = s; }
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
row_argmax_kernel(const T* __restrict__ logits, int64_t row_stride, int N, int V, const int32_t* __restrict__ n_rows,
                  int chunk_elems, int chunks, float* __restrict__ pval, int* __restrict__ pid) {
    constexpr int VN = Vec16<T>::N;
    const int row = blockIdx.x / chunks, chunk = blockIdx.x % chunks;
    if (row % N >= n_rows[row / N]) return;  // padding row: never read
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const T* x = logits + static_cast<int64_t>(row) * row_stride;
    const int begin = chunk * chunk_elems;
    const int end = min(V, begin + chunk_elems);
    const int vec_end = begin + ((end - begin) / VN) * VN;

    float bv = -CUDART_INF_F;
    int bi = 0x7fffffff;
    constexpr int kStep = kThreads * VN;
    for (int it = begin + tid * VN; it < vec_end; it += kUnroll * kStep) {
        float vals[kUnroll][VN];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int id0 = it + u * kStep;
            if (id0 < vec_end) Vec16<T>::load(x + id0, vals[u]);
            else {
#pragma unroll
                for (int e = 0; e < VN; ++e) vals[u][e] = -CUDART_INF_F;
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
#pragma unroll
            for (int e = 0; e < VN; ++e)
                if (vals[u][e] > bv) { bv = vals[u][e]; bi = it + u * kStep + e; }  // ids ascend: first maximum kept
        }
    }
    if (tid < end - vec_end) {
        const float v = Vec16<T>::scalar(x + vec_end + tid);
        if (beats(v, vec_end + tid, bv, bi)) { bv = v; bi = vec_end + tid; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        const float v2 = __shfl_xor_sync(kFull, bv, o);
        const int i2 = __shfl_xor_sync(kFull, bi, o);
        if (beats(v2, i2, bv, bi)) { bv = v2; bi = i2; }
    }
    __shared__ float sm_v[kWarps];
    __shared__ int sm_i[kWarps];
    if (lane == 0) { sm_v[warp] = bv; sm_i[warp] = bi; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < kWarps; ++w)
            if (beats(sm_v[w], sm_i[w], bv, bi)) { bv = sm_v[w]; bi = sm_i[w]; }
        pval[static_cast<size_t>(row) * chunks + chunk] = bv;
        pid[static_cast<size_t>(row) * chunks + chunk] = bi;
    }
}

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

int pick_chunk(int64_t rows, int V, int lo, int hi) {
    // Aim at ~16 CTAs per SM over the whole pass (148 SMs) so that the tail wave stays short,
    // but never less than `lo` elements per CTA (per-CTA reduction overhead) nor more than `hi`.
    const int64_t total = rows * static_cast<int64_t>(V);
    int64_t c = (total / 2368 + 2047) / 2048 * 2048;
    if (c < lo) c = lo;
    if (c > hi) c = hi;
    return static_cast<int>(c);
}

}  // namespace

BuildPartialLayout build_partial_layout(int R, int L, int V, int K) {
    BuildPartialLayout lay;
    const int64_t rows = static_cast<int64_t>(R) * L;
    lay.chunk_elems = pick_chunk(rows, V, 4096, 65536);
    lay.chunks = (V + lay.chunk_elems - 1) / lay.chunk_elems;
    const size_t n = static_cast<size_t>(rows) * lay.chunks;
    lay.off_m = 0;
    lay.off_s = align_up(lay.off_m + n * 4, 256);
    lay.off_val = align_up(lay.off_s + n * 4, 256);
    lay.off_id = align_up(lay.off_val + n * K * 4, 256);
    lay.total = align_up(lay.off_id + n * K * 4, 256);
    return lay;
}

ArgmaxLayout argmax_layout(int rows, int V) {
    ArgmaxLayout lay;
    lay.chunk_elems = pick_chunk(rows, V, 8192, 65536);
    lay.chunks = (V + lay.chunk_elems - 1) / lay.chunk_elems;
    const size_t n = static_cast<size_t>(rows) * lay.chunks;
    lay.off_val = 0;
    lay.off_id = align_up(n * 4, 256);
    lay.total = align_up(lay.off_id + n * 4, 256);
    return lay;
}

cudaError_t launch_logits_topk(const void* logits, int dt, int64_t row_stride, int rows, int V, int K,
                               const BuildPartialLayout& lay, void* ws, cudaStream_t st) {
    char* w = static_cast<char*>(ws);
    float* pm = reinterpret_cast<float*>(w + lay.off_m);
    float* ps = reinterpret_cast<float*>(w + lay.off_s);
    float* pval = reinterpret_cast<float*>(w + lay.off_val);
    int* pid = reinterpret_cast<int*>(w + lay.off_id);
    const unsigned grid = static_cast<unsigned>(lay.chunks) * rows;
    if (dt == DDTREE_F32)
        logits_topk_kernel<float><<<grid, kThreads, 0, st>>>(static_cast<const float*>(logits), row_stride, V, K,
                                                            lay.chunk_elems, lay.chunks, pm, ps, pval, pid);
    else
        logits_topk_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(static_cast<const __nv_bfloat16*>(logits),
                                                                    row_stride, V, K, lay.chunk_elems, lay.chunks,
                                                                    pm, ps, pval, pid);
    return cudaGetLastError();
}

cudaError_t launch_row_argmax(const void* logits, int dt, int64_t row_stride, int R, int N, int V,
                              const int32_t* n_rows, const ArgmaxLayout& lay, void* ws, cudaStream_t st) {
    char* w = static_cast<char*>(ws);
    float* pval = reinterpret_cast<float*>(w + lay.off_val);
    int* pid = reinterpret_cast<int*>(w + lay.off_id);
    const unsigned grid = static_cast<unsigned>(lay.chunks) * R * N;
    if (dt == DDTREE_F32)
        row_argmax_kernel<float><<<grid, kThreads, 0, st>>>(static_cast<const float*>(logits), row_stride, N, V,
                                                           n_rows, lay.chunk_elems, lay.chunks, pval, pid);
    else
        row_argmax_kernel<__nv_bfloat16><<<grid, kThreads, 0, st>>>(static_cast<const __nv_bfloat16*>(logits),
                                                                   row_stride, N, V, n_rows, lay.chunk_elems,
                                                                   lay.chunks, pval, pid);
    return cudaGetLastError();
}

}  // namespace ddtree

// Vocabulary-wide passes over logits rows (HBM-bound):
//   logits_stats_kernel -- per (row, tile): max and sum of exponentials, plus per-warp and per-thread
//                          maxima from which the K best tokens are recovered (Sections 3 and 4.3:
//                          q_i = softmax(l_i), tokens ranked by probability).
//   row_argmax_kernel   -- per (row, chunk): maximum and the lowest id attaining it (the greedy
//                          decoding rule of Section 4.4).
//   row_weight_sums_kernel / row_sample_kernel -- the temperature-based decoding rule of Section 4.4:
//                          per (row, chunk) sums of fixed-point softmax weights, then the inverse-CDF
//                          draw of every row's token.
// All read each element once per pass with 16-byte loads; chunk partials are merged by the kernels in
// tree_build.cu / accept_walk.cu.
#include "common.cuh"
#include <cooperative_groups.h>
#include <math_constants.h>

namespace ddtree {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kUnroll = 4;
constexpr int kPerThread = kTopkChunk / kThreads;  // elements per thread of a drafter tile (32)
static_assert(kThreads == kTopkThreads, "tile ownership is defined for 256-thread CTAs");
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

__device__ __forceinline__ unsigned orderable(float f) {
    const unsigned u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float from_orderable(unsigned k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ float ex2_approx(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ void online_merge(float& m, float& s, float m2, float s2) {
    const float M = fmaxf(m, m2);
    if (M == -CUDART_INF_F) { m = M; s = 0.f; return; }
    s = s * exp2f((m - M) * kLog2e) + s2 * exp2f((m2 - M) * kLog2e);
    m = M;
}

// Drafter logits pass.  A tile is kTopkChunk consecutive elements of one row; thread t of the CTA
// owns the 16-byte vectors v*256 + t (v = 0..) of the tile.  The pass is a pure streaming reduction:
// per tile it writes max and sum of exponentials, per warp the warp's maximum, and per thread the
// maximum of the thread's 32 elements.  The top-K of a row is recovered afterwards from those thread
// maxima (tree_build.cu): the K-th largest thread maximum bounds the K-th largest element from
// below, so only about K threads' elements are ever looked at again.
//
// One CTA per tile and no staging: every thread issues all the 16-byte loads of its 32 elements at
// once (128 bytes in flight per thread), and occupancy, not a software pipeline, keeps the memory
// system busy.  (A persistent version that streamed tiles through shared memory with cp.async
// double buffering reached 4.66 TB/s on 156 MB; this one 5.3 TB/s.)
template <typename T>
__global__ void __launch_bounds__(kThreads, 6)
logits_stats_kernel(const T* __restrict__ logits, int64_t row_stride, int V, int chunks,
                           float* __restrict__ pm, float* __restrict__ ps, float* __restrict__ tmax,
                           float* __restrict__ wmax) {
    constexpr int VN = Vec16<T>::N;
    constexpr int NV = kPerThread / VN;
    __shared__ float sm_m[kWarps], sm_s[kWarps];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_wait();
    const int tile = blockIdx.x;
    const int row = tile / chunks, begin = (tile % chunks) * kTopkChunk;
    const T* x = logits + static_cast<int64_t>(row) * row_stride;
    float val[NV][VN];
#pragma unroll
    for (int v = 0; v < NV; ++v) {
        const int id0 = begin + (v * kThreads + tid) * VN;
        if (id0 + VN <= V) Vec16<T>::load(x + id0, val[v]);
        else {  // ragged end of the row: element-wise, padded with -inf
#pragma unroll
            for (int e = 0; e < VN; ++e) val[v][e] = id0 + e < V ? Vec16<T>::scalar(x + id0 + e) : -CUDART_INF_F;
        }
    }
    float m4[4] = {-CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F, -CUDART_INF_F};
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VN; ++e) m4[e & 3] = fmaxf(m4[e & 3], val[v][e]);
    const float m = fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]));
    tmax[static_cast<size_t>(tile) * kThreads + tid] = m;
    // exponentials relative to the warp maximum, four partial sums to keep the add chain short
    const float wm = from_orderable(__reduce_max_sync(kFull, orderable(m)));
    const float mm = wm == -CUDART_INF_F ? 0.f : wm * kLog2e;
    float s4[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
    for (int v = 0; v < NV; ++v)
#pragma unroll
        for (int e = 0; e < VN; ++e) s4[e & 3] += ex2_approx(fmaf(val[v][e], kLog2e, -mm));
    float s = (s4[0] + s4[1]) + (s4[2] + s4[3]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(kFull, s, o);
    if (lane == 0) { sm_m[warp] = wm; sm_s[warp] = s; wmax[static_cast<size_t>(tile) * kWarps + warp] = wm; }
    __syncthreads();
    if (tid == 0) {
        float M = sm_m[0], S = sm_s[0];
#pragma unroll
        for (int w = 1; w < kWarps; ++w) online_merge(M, S, sm_m[w], sm_s[w]);
        pm[tile] = M;
        ps[tile] = S;
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
row_argmax_kernel(const T* __restrict__ logits, int64_t row_stride, int N, int V, const int32_t* __restrict__ n_rows,
                  int chunk_elems, int chunks, float* __restrict__ pval, int* __restrict__ pid) {
    constexpr int VN = Vec16<T>::N;
    pdl_wait();
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

// ---- temperature-based decoding rule ---------------------------------------------------------------
// The target's choice at a row is a draw from softmax(x / T) (Section 4.4).  The draw is defined on integers so
// that it does not depend on the order of any sum: token v has the weight
//     W_v = floor(2^40 * e_v),  e_v = 2^((x_v - max x) * c),  c = float32(log2(e) / T),
// with e_v evaluated in float32, one rounding per operation: t = (x_v - max) * c; n = t rounded to the nearest
// integer by adding 1.5 * 2^23 (the integer is then read from the sum's bit pattern); f = t - n in [-1/2, 1/2];
// a degree-5 polynomial p for 2^f in Horner form, multiply then add; W_v = significand of p shifted by its
// exponent + n + 17; tokens with t < -40 weigh nothing.  The row's random input k (32 bits) selects the
// smallest v whose inclusive prefix sum exceeds floor(total * k / 2^32).  No instruction of the weight goes
// through the conversion unit (16 results per clock and SM): rounding and the float -> fixed-point step are
// integer operations on bit patterns.
__device__ __forceinline__ unsigned long long sample_weight(float x, float m, float c) {
    const float t = __fmul_rn(__fsub_rn(x, m), c);
    if (!(t >= -40.f)) return 0ull;  // also -inf and NaN
    const float r = __fadd_rn(t, 12582912.f);
    const int n = static_cast<int>(__float_as_uint(r)) - 0x4B400000;
    const float f = __fsub_rn(t, __fsub_rn(r, 12582912.f));
    float acc = 0.00132647273f;
    acc = __fadd_rn(__fmul_rn(acc, f), 0.00967151299f);
    acc = __fadd_rn(__fmul_rn(acc, f), 0.0555073358f);
    acc = __fadd_rn(__fmul_rn(acc, f), 0.240222424f);
    acc = __fadd_rn(__fmul_rn(acc, f), 0.693147004f);
    acc = __fadd_rn(__fmul_rn(acc, f), 1.0f);
    const unsigned bits = __float_as_uint(acc);
    const unsigned sig = (bits & 0x7FFFFFu) | 0x800000u;            // p = sig * 2^(e - 23), e in {-1, 0}
    // floor(p * 2^n * 2^40) = floor(sig * 2^(e + 17 + n)): a constant left shift, then a right shift by -(e + n) in [0, 41]
    const int down = 127 - static_cast<int>(bits >> 23) - n;
    return (static_cast<unsigned long long>(sig) << 17) >> down;
}

// w[0] + ... + w[e]
template <int VN>
__device__ __forceinline__ unsigned long long prefix_to(const unsigned long long (&w)[VN], int e) {
    unsigned long long s = 0;
#pragma unroll
    for (int i = 0; i < VN; ++i)
        if (i <= e) s += w[i];
    return s;
}

// Row maximum from the arg-max pass's chunk partials (every thread reads them all: there are few).
__device__ __forceinline__ float row_max_of(const float* __restrict__ pval, int chunks) {
    float m = -CUDART_INF_F;
    for (int c = 0; c < chunks; ++c) m = fmaxf(m, pval[c]);
    return m;
}

__device__ __forceinline__ unsigned long long block_sum_u64(unsigned long long v, unsigned long long* sm) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (lane == 0) sm[warp] = v;
    __syncthreads();
    unsigned long long t = 0;
    for (int w = 0; w < kWarps; ++w) t += sm[w];
    return t;
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
row_weight_sums_kernel(const T* __restrict__ logits, int64_t row_stride, int N, int V, const int32_t* __restrict__ n_rows,
                       int chunk_elems, int chunks, float c, const float* __restrict__ pval,
                       unsigned long long* __restrict__ psum) {
    constexpr int VN = Vec16<T>::N;
    pdl_wait();
    const int row = blockIdx.x / chunks, chunk = blockIdx.x % chunks;
    if (row % N >= n_rows[row / N]) return;  // padding row: never read
    const int tid = threadIdx.x;
    const float m = row_max_of(pval + static_cast<size_t>(row) * chunks, chunks);
    const T* x = logits + static_cast<int64_t>(row) * row_stride;
    const int begin = chunk * chunk_elems;
    const int end = min(V, begin + chunk_elems);
    const int vec_end = begin + ((end - begin) / VN) * VN;
    unsigned long long acc = 0;
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
        for (int u = 0; u < kUnroll; ++u)
#pragma unroll
            for (int e = 0; e < VN; ++e) acc += sample_weight(vals[u][e], m, c);
    }
    if (tid < end - vec_end) acc += sample_weight(Vec16<T>::scalar(x + vec_end + tid), m, c);
    __shared__ unsigned long long sm[kWarps];
    const unsigned long long total = block_sum_u64(acc, sm);
    if (tid == 0) psum[static_cast<size_t>(row) * chunks + chunk] = total;
}

// One CTA per row: find the chunk the threshold falls into from the chunk sums, then the token inside that chunk.
// The chunk is walked in rounds of 256 x (elements per 16-byte vector) consecutive tokens: every thread weighs
// its vector, a block scan of the thread sums tells whether the threshold falls into this round and into which
// thread's vector; otherwise the round's total is taken off the threshold.
template <typename T>
__global__ void __launch_bounds__(kThreads)
row_sample_kernel(const T* __restrict__ logits, int64_t row_stride, int N, int V, const int32_t* __restrict__ n_rows,
                  int chunk_elems, int chunks, float c, const float* __restrict__ pval,
                  const unsigned long long* __restrict__ psum, const uint32_t* __restrict__ row_uniform,
                  int32_t* __restrict__ token) {
    constexpr int VN = Vec16<T>::N;
    pdl_wait();
    const int row = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (row % N >= n_rows[row / N]) {
        if (tid == 0) token[row] = -1;
        return;
    }
    const float m = row_max_of(pval + static_cast<size_t>(row) * chunks, chunks);
    const unsigned long long* ps = psum + static_cast<size_t>(row) * chunks;
    unsigned long long total = 0;
    for (int k = 0; k < chunks; ++k) total += ps[k];
    if (total == 0) {  // no finite maximum in the row: nothing to draw from
        if (tid == 0) token[row] = -1;
        return;
    }
    const unsigned long long u = row_uniform[row];
    unsigned long long thr = (__umul64hi(total, u) << 32) | ((total * u) >> 32);  // floor(total * u / 2^32) < total
    int chunk = 0;
    while (chunk + 1 < chunks && thr >= ps[chunk]) thr -= ps[chunk++];  // thr is now relative to the chunk's first token
    const T* x = logits + static_cast<int64_t>(row) * row_stride;
    const int end = min(V, (chunk + 1) * chunk_elems);
    __shared__ unsigned long long warp_total[kWarps];
    for (int base = chunk * chunk_elems; base < end; base += kThreads * VN) {  // chunk starts are multiples of 2048
        const int id0 = base + tid * VN;
        float vals[VN];
        if (id0 + VN <= end) {
            Vec16<T>::load(x + id0, vals);
        } else {
#pragma unroll
            for (int e = 0; e < VN; ++e) vals[e] = id0 + e < end ? Vec16<T>::scalar(x + id0 + e) : -CUDART_INF_F;
        }
        unsigned long long w[VN], mine = 0;
#pragma unroll
        for (int e = 0; e < VN; ++e) { w[e] = sample_weight(vals[e], m, c); mine += w[e]; }
        unsigned long long incl = mine;  // inclusive scan over the warp, then over the warps
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned long long up = __shfl_up_sync(kFull, incl, o);
            if (lane >= o) incl += up;
        }
        if (lane == 31) warp_total[warp] = incl;
        __syncthreads();
        unsigned long long round_total = 0;
        for (int k = 0; k < kWarps; ++k) {
            if (k < warp) incl += warp_total[k];
            round_total += warp_total[k];
        }
        if (thr < round_total) {  // the same for every thread
            unsigned long long acc = incl - mine;
            if (acc <= thr && thr < incl) {  // exactly one thread: the inclusive sums never decrease
                int found = id0 + VN - 1;
#pragma unroll
                for (int e = VN - 1; e >= 0; --e)
                    if (acc + prefix_to<VN>(w, e) > thr) found = id0 + e;
                token[row] = found;
            }
            return;
        }
        thr -= round_total;
        __syncthreads();  // warp_total is rewritten in the next round
    }
}


// ---- the sampled walk, lazily ----------------------------------------------------------------------------------
// The walk only ever asks for the target's choice at the rows it stands on: the root, then one accepted node
// per step, at most L + 1 rows of a request (Section 4.4).  Instead of weighing every row of every request,
// a cluster of kWalkCtas CTAs per request follows the walk: at each visited row every CTA stages its slice of
// the row's logits in shared memory (one read of the row), the CTAs exchange slice maxima and slice weight
// sums through distributed shared memory, the CTA whose slice holds the threshold finds the token, and all of
// them take the walk's step.  The draw is the one ddtree_accept_sampled defines (fixed-point weights relative
// to the row maximum, threshold floor(total * k / 2^32), smallest token whose inclusive prefix sum exceeds
// it): integer sums, so the partition into slices and threads does not matter.
constexpr int kWalkCtas = 8;
constexpr int kWalkThreads = 512;
constexpr int kWalkWarps = kWalkThreads / 32;
constexpr int kWalkMaxSlice = 56 * 1024;  // fp32 elements of one CTA's slice that fit its shared memory

struct WalkShared {
    float cmax;                          // this CTA's slice maximum (read by the other CTAs of the cluster)
    unsigned long long csum;             // this CTA's slice weight sum
    int ctok;                            // the drawn token, written by the CTA whose slice holds the threshold
    float wmax[kWalkWarps];
    unsigned long long wsum[kWalkWarps];
    int found;
    int token[kMaxN];
    short parent[kMaxN];
};

template <typename T>
__global__ void __launch_bounds__(kWalkThreads, 1)
sampled_walk_kernel(const T* __restrict__ logits, int64_t row_stride, int N, int V, int L, int slice,
                    const int32_t* __restrict__ n_rows, float c, const uint32_t* __restrict__ row_uniform,
                    const int32_t* __restrict__ node_token, const int32_t* __restrict__ node_parent,
                    int32_t* __restrict__ accept_len, int32_t* __restrict__ accept_nodes,
                    int32_t* __restrict__ accept_tokens, int32_t* __restrict__ bonus_token) {
    namespace cg = cooperative_groups;
    constexpr int VN = Vec16<T>::N;
    extern __shared__ __align__(16) unsigned char walk_smem[];
    WalkShared& sh = *reinterpret_cast<WalkShared*>(walk_smem);
    float* xs = reinterpret_cast<float*>(walk_smem + ((sizeof(WalkShared) + 15) / 16) * 16);  // the staged slice, fp32
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = static_cast<int>(cluster.block_rank());
    const int r = blockIdx.x / kWalkCtas, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_wait();
    const int n = min(n_rows[r], N);
    const size_t o = static_cast<size_t>(r) * N;
    for (int row = tid; row < n; row += kWalkThreads) {
        sh.token[row] = node_token[o + row];
        sh.parent[row] = static_cast<short>(node_parent[o + row]);
    }
    const int begin = rank * slice, end = min(V, begin + slice);  // my tokens (begin is a multiple of 8)
    const int count = max(0, end - begin);
    const int per = ((slice + kWalkThreads - 1) / kWalkThreads) | 1;  // tokens per thread in the scan; odd: no bank conflicts
    const WalkShared* peer[kWalkCtas];
#pragma unroll
    for (int k = 0; k < kWalkCtas; ++k) peer[k] = cluster.map_shared_rank(&sh, k);
    __syncthreads();

    int cur = 0, len = 0, tok = -1;
    for (;;) {
        // ---- 1. stage my slice of row `cur`, slice maximum ------------------------------------------------
        const T* x = logits + static_cast<int64_t>(o + cur) * row_stride + begin;
        float m = -CUDART_INF_F;
        const int vec_count = (count / VN) * VN;
        for (int i = tid * VN; i < vec_count; i += kWalkThreads * VN) {
            float v[VN];
            Vec16<T>::load(x + i, v);
#pragma unroll
            for (int e = 0; e < VN; ++e) { xs[i + e] = v[e]; m = fmaxf(m, v[e]); }
        }
        for (int i = vec_count + tid; i < count; i += kWalkThreads) {
            const float v = Vec16<T>::scalar(x + i);
            xs[i] = v;
            m = fmaxf(m, v);
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) m = fmaxf(m, __shfl_xor_sync(kFull, m, d));
        if (lane == 0) sh.wmax[warp] = m;
        __syncthreads();
        if (tid == 0) {
            float mm = sh.wmax[0];
            for (int k = 1; k < kWalkWarps; ++k) mm = fmaxf(mm, sh.wmax[k]);
            sh.cmax = mm;
        }
        cluster.sync();
        float row_max = -CUDART_INF_F;
#pragma unroll
        for (int k = 0; k < kWalkCtas; ++k) row_max = fmaxf(row_max, peer[k]->cmax);

        // ---- 2. weights of my slice: thread t owns tokens [t * per, (t + 1) * per) of it -----------------------
        const int t0 = min(count, tid * per), t1 = min(count, t0 + per);
        unsigned long long mine = 0;
        for (int i = t0; i < t1; ++i) mine += sample_weight(xs[i], row_max, c);
        unsigned long long incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const unsigned long long up = __shfl_up_sync(kFull, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) sh.wsum[warp] = incl;
        __syncthreads();
        unsigned long long before_me = 0, slice_total = 0;
        for (int k = 0; k < kWalkWarps; ++k) {
            if (k < warp) before_me += sh.wsum[k];
            slice_total += sh.wsum[k];
        }
        incl += before_me;
        if (tid == 0) { sh.csum = slice_total; sh.ctok = -1; }
        cluster.sync();
        unsigned long long total = 0, before_slice = 0;
#pragma unroll
        for (int k = 0; k < kWalkCtas; ++k) {
            const unsigned long long sk = peer[k]->csum;
            if (k < rank) before_slice += sk;
            total += sk;
        }

        // ---- 3. the draw: the thread whose tokens hold the threshold names the token ---------------------------
        if (total > 0) {  // else: no finite maximum in the row, nothing to draw from (token -1, the walk stops)
            const unsigned long long u = row_uniform[o + cur];
            const unsigned long long thr = (__umul64hi(total, u) << 32) | ((total * u) >> 32);  // floor(total * u / 2^32) < total
            const unsigned long long lo = before_slice + (incl - mine), hi = before_slice + incl;
            if (lo <= thr && thr < hi) {  // exactly one thread of the cluster
                unsigned long long acc = lo;
                int found = t1 - 1;
                for (int i = t0; i < t1; ++i) {
                    acc += sample_weight(xs[i], row_max, c);
                    if (acc > thr) { found = i; break; }
                }
                sh.ctok = begin + found;
            }
        }
        cluster.sync();
        tok = -1;
#pragma unroll
        for (int k = 0; k < kWalkCtas; ++k) tok = max(tok, peer[k]->ctok);

        // ---- 4. the walk's step (every CTA takes it; rank 0 writes) -------------------------------------------
        if (len >= L || tok < 0) break;
        if (tid == 0) sh.found = 0x7fffffff;
        __syncthreads();
        for (int j = cur + 1 + tid; j < n; j += kWalkThreads)   // children have larger rows; siblings carry distinct tokens
            if (sh.parent[j] == cur && sh.token[j] == tok) atomicMin(&sh.found, j);
        __syncthreads();
        const int found = sh.found;
        if (found == 0x7fffffff) break;
        if (rank == 0 && tid == 0) {
            accept_nodes[static_cast<size_t>(r) * L + len] = found;
            accept_tokens[static_cast<size_t>(r) * L + len] = tok;
        }
        cur = found;
        ++len;
        __syncthreads();  // sh.found and the staged slice are rewritten in the next round
    }
    if (rank == 0) {
        for (int k = len + tid; k < L; k += kWalkThreads) {
            accept_nodes[static_cast<size_t>(r) * L + k] = -1;
            accept_tokens[static_cast<size_t>(r) * L + k] = -1;
        }
        if (tid == 0) {
            accept_len[r] = len;
            bonus_token[r] = tok;
        }
    }
    cluster.sync();  // no CTA leaves while a neighbour may still read its shared memory
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
    (void)K;
    (void)pick_chunk;
    BuildPartialLayout lay;
    const int64_t rows = static_cast<int64_t>(R) * L;
    lay.chunk_elems = kTopkChunk;
    lay.chunks = (V + lay.chunk_elems - 1) / lay.chunk_elems;
    const size_t n = static_cast<size_t>(rows) * lay.chunks;
    lay.off_m = 0;
    lay.off_s = align_up(lay.off_m + n * 4, 256);
    lay.off_tmax = align_up(lay.off_s + n * 4, 256);
    lay.off_wmax = align_up(lay.off_tmax + n * kThreads * 4, 256);
    lay.total = align_up(lay.off_wmax + n * kWarps * 4, 256);
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

cudaError_t launch_logits_stats(const void* logits, int dt, int64_t row_stride, int rows, int V,
                                const BuildPartialLayout& lay, void* ws, cudaStream_t st) {
    char* w = static_cast<char*>(ws);
    float* pm = reinterpret_cast<float*>(w + lay.off_m);
    float* ps = reinterpret_cast<float*>(w + lay.off_s);
    float* tmax = reinterpret_cast<float*>(w + lay.off_tmax);
    float* wmax = reinterpret_cast<float*>(w + lay.off_wmax);
    const int tiles = lay.chunks * rows;
    if (dt == DDTREE_F32)
        return launch_pdl(logits_stats_kernel<float>, dim3(tiles), dim3(kThreads), 0, st,
                          static_cast<const float*>(logits), row_stride, V, lay.chunks, pm, ps, tmax, wmax);
    return launch_pdl(logits_stats_kernel<__nv_bfloat16>, dim3(tiles), dim3(kThreads), 0, st,
                      static_cast<const __nv_bfloat16*>(logits), row_stride, V, lay.chunks, pm, ps, tmax, wmax);
}

cudaError_t launch_row_argmax(const void* logits, int dt, int64_t row_stride, int R, int N, int V,
                              const int32_t* n_rows, const ArgmaxLayout& lay, void* ws, cudaStream_t st) {
    char* w = static_cast<char*>(ws);
    float* pval = reinterpret_cast<float*>(w + lay.off_val);
    int* pid = reinterpret_cast<int*>(w + lay.off_id);
    const unsigned grid = static_cast<unsigned>(lay.chunks) * R * N;
    if (dt == DDTREE_F32)
        return launch_pdl(row_argmax_kernel<float>, dim3(grid), dim3(kThreads), 0, st, static_cast<const float*>(logits),
                          row_stride, N, V, n_rows, lay.chunk_elems, lay.chunks, pval, pid);
    return launch_pdl(row_argmax_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, st,
                      static_cast<const __nv_bfloat16*>(logits), row_stride, N, V, n_rows, lay.chunk_elems, lay.chunks,
                      pval, pid);
}

SampleLayout sample_layout(int rows, int V) {
    SampleLayout lay;
    lay.a = argmax_layout(rows, V);
    lay.off_sum = lay.a.total;
    lay.off_tok = align_up(lay.off_sum + static_cast<size_t>(rows) * lay.a.chunks * 8, 256);
    lay.total = align_up(lay.off_tok + static_cast<size_t>(rows) * 4, 256);
    return lay;
}

cudaError_t launch_row_sample(const void* logits, int dt, int64_t row_stride, int R, int N, int V, const int32_t* n_rows,
                              float log2e_over_t, const uint32_t* row_uniform, const SampleLayout& lay, void* ws,
                              cudaStream_t st) {
    char* w = static_cast<char*>(ws);
    const float* pval = reinterpret_cast<const float*>(w + lay.a.off_val);
    unsigned long long* psum = reinterpret_cast<unsigned long long*>(w + lay.off_sum);
    int32_t* token = reinterpret_cast<int32_t*>(w + lay.off_tok);
    const unsigned rows = static_cast<unsigned>(R) * N;
    const unsigned grid = static_cast<unsigned>(lay.a.chunks) * rows;
    cudaError_t e;
    if (dt == DDTREE_F32) {
        e = launch_pdl(row_weight_sums_kernel<float>, dim3(grid), dim3(kThreads), 0, st, static_cast<const float*>(logits),
                       row_stride, N, V, n_rows, lay.a.chunk_elems, lay.a.chunks, log2e_over_t, pval, psum);
        if (e != cudaSuccess) return e;
        return launch_pdl(row_sample_kernel<float>, dim3(rows), dim3(kThreads), 0, st, static_cast<const float*>(logits),
                          row_stride, N, V, n_rows, lay.a.chunk_elems, lay.a.chunks, log2e_over_t, pval, psum, row_uniform, token);
    }
    e = launch_pdl(row_weight_sums_kernel<__nv_bfloat16>, dim3(grid), dim3(kThreads), 0, st,
                   static_cast<const __nv_bfloat16*>(logits), row_stride, N, V, n_rows, lay.a.chunk_elems, lay.a.chunks,
                   log2e_over_t, pval, psum);
    if (e != cudaSuccess) return e;
    return launch_pdl(row_sample_kernel<__nv_bfloat16>, dim3(rows), dim3(kThreads), 0, st,
                      static_cast<const __nv_bfloat16*>(logits), row_stride, N, V, n_rows, lay.a.chunk_elems, lay.a.chunks,
                      log2e_over_t, pval, psum, row_uniform, token);
}

bool sampled_walk_fits(int V) { return (V + kWalkCtas - 1) / kWalkCtas <= kWalkMaxSlice - 8; }

template <typename T>
static cudaError_t launch_sampled_walk_t(const T* logits, int64_t row_stride, int R, int N, int V, int L, const int32_t* n_rows,
                                         float c, const uint32_t* row_uniform, const int32_t* node_token, const int32_t* node_parent,
                                         int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens, int32_t* bonus_token,
                                         cudaStream_t st) {
    const int slice = ((V + kWalkCtas - 1) / kWalkCtas + 7) / 8 * 8;  // slices start on 16-byte boundaries
    const size_t smem = ((sizeof(WalkShared) + 15) / 16) * 16 + static_cast<size_t>(slice) * 4;
    cudaError_t e = cudaFuncSetAttribute(sampled_walk_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(static_cast<unsigned>(R) * kWalkCtas);
    cfg.blockDim = dim3(kWalkThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kWalkCtas;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, sampled_walk_kernel<T>, logits, row_stride, N, V, L, slice, n_rows, c, row_uniform, node_token,
                              node_parent, accept_len, accept_nodes, accept_tokens, bonus_token);
}

cudaError_t launch_sampled_walk(const void* logits, int dt, int64_t row_stride, int R, int N, int V, int L, const int32_t* n_rows,
                                float log2e_over_t, const uint32_t* row_uniform, const int32_t* node_token,
                                const int32_t* node_parent, int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                                int32_t* bonus_token, cudaStream_t st) {
    if (dt == DDTREE_F32)
        return launch_sampled_walk_t(static_cast<const float*>(logits), row_stride, R, N, V, L, n_rows, log2e_over_t, row_uniform,
                                     node_token, node_parent, accept_len, accept_nodes, accept_tokens, bonus_token, st);
    return launch_sampled_walk_t(static_cast<const __nv_bfloat16*>(logits), row_stride, R, N, V, L, n_rows, log2e_over_t,
                                 row_uniform, node_token, node_parent, accept_len, accept_nodes, accept_tokens, bonus_token, st);
}

}  // namespace ddtree

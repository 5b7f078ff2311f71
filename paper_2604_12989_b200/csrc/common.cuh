// Shared declarations of the DDTree CUDA library (internal; the public surface is include/ddtree.h).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>
#include "ddtree.h"

namespace ddtree {

constexpr int kMaxK = 32;     // tokens kept per position
constexpr int kMaxL = 32;     // draft positions
constexpr int kMaxB = 1024;   // node budget
constexpr int kMaxN = kMaxB + 1;

// Records a message for ddtree_last_error() and returns `code`.
int fail(int code, const char* fmt, ...);

// Drafter logits pass: a tile is kTopkChunk consecutive elements of one logits row, reduced by a
// CTA of kTopkThreads threads; thread t owns the 16-byte vectors v*kTopkThreads + t of the tile.
// Per tile the pass leaves max and sum of exp(x - max), per warp and per thread the maximum of
// their elements.
constexpr int kTopkChunk = 8192;
constexpr int kTopkThreads = 256;
struct BuildPartialLayout {
    int chunks;        // tiles per row
    int chunk_elems;   // = kTopkChunk
    size_t off_m, off_s, off_tmax, off_wmax, total;  // byte offsets into the workspace
};
BuildPartialLayout build_partial_layout(int R, int L, int V, int K);

struct ArgmaxLayout {
    int chunks;
    int chunk_elems;
    size_t off_val, off_id, total;
};
ArgmaxLayout argmax_layout(int rows, int V);

// Kernel launchers (each enqueues on `st` and returns cudaGetLastError()).
cudaError_t launch_logits_stats(const void* logits, int dt, int64_t row_stride, int rows, int V,
                                const BuildPartialLayout& lay, void* ws, cudaStream_t st);
cudaError_t launch_tree_build(int R, int L, int V, int K, int B, const BuildPartialLayout& lay, const void* ws,
                              const void* logits, int dt, int64_t row_stride,
                              const int32_t* root_token, const int32_t* prefix_len,
                              int32_t* n_rows, int32_t* node_token, int32_t* node_parent, int32_t* node_depth,
                              int32_t* position_ids, uint32_t* anc_mask, int32_t* first_child,
                              int32_t* child_count, float* node_logprob, int32_t* topk_token,
                              float* topk_logprob, cudaStream_t st);
cudaError_t launch_row_argmax(const void* logits, int dt, int64_t row_stride, int R, int N, int V,
                              const int32_t* n_rows, const ArgmaxLayout& lay, void* ws, cudaStream_t st);
// `choice`: NULL = the arg-max of the chunk partials in `ws` is the target's choice at a row; else [R, N] tokens.
cudaError_t launch_accept_walk(int R, int N, int L, const ArgmaxLayout& lay, const void* ws, const int32_t* choice,
                               const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows,
                               int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                               int32_t* bonus_token, int32_t* node_argmax, cudaStream_t st);

// Temperature-based decoding rule: workspace = the arg-max partials, then per (row, chunk) weight sums and the
// sampled token of every row.
struct SampleLayout {
    ArgmaxLayout a;
    size_t off_sum, off_tok, total;
};
SampleLayout sample_layout(int rows, int V);
// After launch_row_argmax on the same workspace: draws the token of every row into the workspace's token array.
cudaError_t launch_row_sample(const void* logits, int dt, int64_t row_stride, int R, int N, int V, const int32_t* n_rows,
                              float log2e_over_t, const uint32_t* row_uniform, const SampleLayout& lay, void* ws,
                              cudaStream_t st);

// The sampled walk without the all-rows passes: one cluster of CTAs per request draws the target's choice only at the
// rows the walk stands on (at most L + 1).  `sampled_walk_fits`: whether a row's slice fits a CTA's shared memory.
bool sampled_walk_fits(int V);
cudaError_t launch_sampled_walk(const void* logits, int dt, int64_t row_stride, int R, int N, int V, int L, const int32_t* n_rows,
                                float log2e_over_t, const uint32_t* row_uniform, const int32_t* node_token,
                                const int32_t* node_parent, int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                                int32_t* bonus_token, cudaStream_t st);

// Rotary positional encoding of the tree's Q / K rows, in place (either pointer may be NULL).
cudaError_t launch_rope_tree(void* q, void* k, const int32_t* position_ids, const int32_t* n_rows, int dt, int R, int N,
                             int Hq, int Hkv, int d, double log2_theta, cudaStream_t st);

struct AttnArgs {
    const void *q, *k_cache, *v_cache, *k_tree, *v_tree;
    const int32_t* cu_prefix;
    const uint32_t* anc_mask;
    const int32_t* n_rows;
    void* out;
    float* lse;
    int R, B, N, W, Hq, Hkv, G, d;
    float scale;
    int max_prefix;     // host-side max over requests of P_r
    int64_t total_prefix;
    // rotary variant (ddtree_tree_attention_rope): q and k_tree are rotated on their way into the products
    int rope = 0;
    const int32_t* position_ids = nullptr;
    double rope_log2_theta = 0.0;
};
cudaError_t launch_tree_attention_f32(const AttnArgs& a, cudaStream_t st);

constexpr int kCompactLayersPerLaunch = 64;  // pointer tables travel as kernel parameters (4 x 64 x 8 bytes)
cudaError_t launch_kv_compact(int R, int N, int L, int row_bytes, int layers, const void* const* k_tree,
                              const void* const* v_tree, void* const* k_cache, void* const* v_cache,
                              const int64_t* dst_row, const int32_t* accept_len, const int32_t* accept_nodes,
                              cudaStream_t st);

size_t tree_attention_bf16_workspace(const AttnArgs& a, const int32_t* cu_prefix_host);
// Returns a ddtree_status (descriptor creation can fail with its own message).
int launch_tree_attention_bf16(const AttnArgs& a, const int32_t* cu_prefix_host, void* ws, size_t ws_bytes,
                               cudaStream_t st);

// Device status word (bounded waits report here).
uint32_t* device_status_word();
// One-thread kernel whose bounded wait runs out after `limit` polls and raises the time-out flag.
cudaError_t launch_wait_timeout_selftest(uint32_t limit, cudaStream_t st);
void tree_attention_set_path(int path);
// kernels one bf16 attention call launches for these shapes (attention, + split merge, + rotary table)
int tree_attention_bf16_kernels(const AttnArgs& a);

// ---- programmatic dependent launch ---------------------------------------------------------------
// Every kernel of this library is launched with programmatic stream serialisation: it may be scheduled
// while the kernel before it in the stream drains, which hides most of the launch latency between the
// ~76 small kernels of a round.  In exchange every kernel calls pdl_wait() before it touches global
// memory: that blocks until the preceding kernel has completed and its writes are visible (and is a
// no-op after a normal launch).  No kernel signals early; measured on B200, explicit early triggers
// made the captured round slower.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
#endif

// ---- small device helpers --------------------------------------------------------------------
__device__ __forceinline__ bool beats(float v, int id, float w, int jd) {
    // (value descending, id ascending): does (v,id) rank strictly before (w,jd)?
    return v > w || (v == w && id < jd);
}

}  // namespace ddtree

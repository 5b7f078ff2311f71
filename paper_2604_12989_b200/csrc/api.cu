// extern "C" surface of the library: argument validation, workspace layout, kernel enqueue.
#include "common.cuh"
#include <cstdarg>
#include <cstdio>
#include <cmath>
#include <mutex>

namespace ddtree {

static thread_local char g_err[512] = "";

int fail(int code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

static __device__ uint32_t g_status_word = 0;

uint32_t* device_status_word() {
    uint32_t* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_status_word) != cudaSuccess) return nullptr;
    return p;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
static int elem_size(int dt) { return dt == DDTREE_F32 ? 4 : 2; }

static int check_logits(const char* fn, const void* logits, int dt, int64_t stride, int V) {
    if (!logits) return fail(DDTREE_ERR_INVALID_ARG, "%s: logits is NULL", fn);
    if (dt != DDTREE_F32 && dt != DDTREE_BF16) return fail(DDTREE_ERR_INVALID_ARG, "%s: unknown dtype %d", fn, dt);
    if (stride < V) return fail(DDTREE_ERR_INVALID_ARG, "%s: row_stride_elems %lld < V %d", fn, (long long)stride, V);
    if (!aligned16(logits) || (stride * elem_size(dt)) % 16 != 0)
        return fail(DDTREE_ERR_INVALID_ARG, "%s: logits rows must start on 16-byte boundaries", fn);
    return DDTREE_OK;
}

static int check_build_sizes(const char* fn, int R, int L, int V, int K, int B) {
    if (R < 1 || L < 1 || V < 1 || K < 1 || B < 1)
        return fail(DDTREE_ERR_INVALID_ARG, "%s: R, L, V, K, B must be >= 1 (got %d %d %d %d %d)", fn, R, L, V, K, B);
    if (K > V) return fail(DDTREE_ERR_INVALID_ARG, "%s: K %d > V %d", fn, K, V);
    if (K > kMaxK) return fail(DDTREE_ERR_INVALID_ARG, "%s: K %d > %d", fn, K, kMaxK);
    if (L > kMaxL) return fail(DDTREE_ERR_INVALID_ARG, "%s: L %d > %d", fn, L, kMaxL);
    if (B > kMaxB) return fail(DDTREE_ERR_INVALID_ARG, "%s: B %d > %d", fn, B, kMaxB);
    return DDTREE_OK;
}

}  // namespace ddtree

using namespace ddtree;

extern "C" {

const char* ddtree_status_string(int status) {
    switch (status) {
        case DDTREE_OK: return "ok";
        case DDTREE_ERR_INVALID_ARG: return "invalid argument";
        case DDTREE_ERR_UNSUPPORTED: return "unsupported configuration";
        case DDTREE_ERR_WORKSPACE: return "workspace too small";
        case DDTREE_ERR_CUDA: return "CUDA error";
        case DDTREE_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        default: return "unknown status";
    }
}

const char* ddtree_last_error(void) { return g_err; }

size_t ddtree_build_workspace_bytes(int R, int L, int V, int K, int B) {
    if (check_build_sizes("ddtree_build_workspace_bytes", R, L, V, K, B) != DDTREE_OK) return 0;
    return build_partial_layout(R, L, V, K).total;
}

int ddtree_build(const void* drafter_logits, int dt, int64_t row_stride_elems, int R, int L, int V, int K, int B,
                 const int32_t* root_token, const int32_t* prefix_len, int32_t* n_rows, int32_t* node_token,
                 int32_t* node_parent, int32_t* node_depth, int32_t* position_ids, uint32_t* anc_mask,
                 int32_t* first_child, int32_t* child_count, float* node_logprob, int32_t* topk_token,
                 float* topk_logprob, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    int rc = check_build_sizes("ddtree_build", R, L, V, K, B);
    if (rc) return rc;
    rc = check_logits("ddtree_build", drafter_logits, dt, row_stride_elems, V);
    if (rc) return rc;
    if (!root_token || !prefix_len || !n_rows || !node_token || !node_parent || !node_depth || !position_ids ||
        !anc_mask)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_build: a required pointer is NULL");
    const BuildPartialLayout lay = build_partial_layout(R, L, V, K);
    if (!workspace || !((reinterpret_cast<uintptr_t>(workspace) & 15u) == 0))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_build: workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < lay.total)
        return fail(DDTREE_ERR_WORKSPACE, "ddtree_build: workspace %zu < required %zu bytes", workspace_bytes, lay.total);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = launch_logits_stats(drafter_logits, dt, row_stride_elems, R * L, V, lay, workspace, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_build: logits pass: %s", cudaGetErrorString(e));
    e = launch_tree_build(R, L, V, K, B, lay, workspace, drafter_logits, dt, row_stride_elems, root_token, prefix_len, n_rows, node_token, node_parent,
                          node_depth, position_ids, anc_mask, first_child, child_count, node_logprob, topk_token,
                          topk_logprob, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_build: tree kernel: %s", cudaGetErrorString(e));
    return DDTREE_OK;
}

size_t ddtree_accept_workspace_bytes(int R, int B, int V) {
    if (R < 1 || B < 1 || B > kMaxB || V < 1) return 0;
    return argmax_layout(R * (B + 1), V).total;
}

int ddtree_accept(const void* target_logits, int dt, int64_t row_stride_elems, int R, int B, int V, int L,
                  const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows, int32_t* accept_len,
                  int32_t* accept_nodes, int32_t* accept_tokens, int32_t* bonus_token, int32_t* node_argmax,
                  void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (R < 1 || B < 1 || V < 1 || L < 1)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept: R, B, V, L must be >= 1 (got %d %d %d %d)", R, B, V, L);
    if (B > kMaxB) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept: B %d > %d", B, kMaxB);
    if (L > kMaxL) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept: L %d > %d", L, kMaxL);
    int rc = check_logits("ddtree_accept", target_logits, dt, row_stride_elems, V);
    if (rc) return rc;
    if (!node_token || !node_parent || !n_rows || !accept_len || !accept_nodes || !accept_tokens || !bonus_token)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept: a required pointer is NULL");
    const ArgmaxLayout lay = argmax_layout(R * (B + 1), V);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept: workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < lay.total)
        return fail(DDTREE_ERR_WORKSPACE, "ddtree_accept: workspace %zu < required %zu bytes", workspace_bytes, lay.total);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    cudaError_t e = launch_row_argmax(target_logits, dt, row_stride_elems, R, B + 1, V, n_rows, lay, workspace, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept: argmax pass: %s", cudaGetErrorString(e));
    e = launch_accept_walk(R, B + 1, L, lay, workspace, nullptr, node_token, node_parent, n_rows, accept_len, accept_nodes,
                           accept_tokens, bonus_token, node_argmax, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept: walk kernel: %s", cudaGetErrorString(e));
    return DDTREE_OK;
}

size_t ddtree_accept_sampled_workspace_bytes(int R, int B, int V) {
    if (R < 1 || B < 1 || B > kMaxB || V < 1) return 0;
    return sample_layout(R * (B + 1), V).total;
}

int ddtree_accept_sampled(const void* target_logits, int dt, int64_t row_stride_elems, int R, int B, int V, int L,
                          const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows, float temperature,
                          const uint32_t* row_uniform, int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                          int32_t* bonus_token, int32_t* node_choice, void* workspace, size_t workspace_bytes,
                          void* cuda_stream) {
    if (R < 1 || B < 1 || V < 1 || L < 1)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: R, B, V, L must be >= 1 (got %d %d %d %d)", R, B, V, L);
    if (B > kMaxB) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: B %d > %d", B, kMaxB);
    if (L > kMaxL) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: L %d > %d", L, kMaxL);
    if (V > (1 << 22)) return fail(DDTREE_ERR_UNSUPPORTED, "ddtree_accept_sampled: V %d > 2^22 (64-bit weight sums)", V);
    if (!(temperature > 0.f) || !(temperature <= 3.0e38f))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: temperature must be positive and finite");
    const float c = static_cast<float>(1.4426950408889634 / static_cast<double>(temperature));
    if (!(c <= 3.0e38f)) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: temperature too small");
    int rc = check_logits("ddtree_accept_sampled", target_logits, dt, row_stride_elems, V);
    if (rc) return rc;
    if (!node_token || !node_parent || !n_rows || !row_uniform || !accept_len || !accept_nodes || !accept_tokens || !bonus_token)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: a required pointer is NULL");
    const SampleLayout lay = sample_layout(R * (B + 1), V);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_sampled: workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < lay.total)
        return fail(DDTREE_ERR_WORKSPACE, "ddtree_accept_sampled: workspace %zu < required %zu bytes", workspace_bytes, lay.total);
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (!node_choice && sampled_walk_fits(V)) {
        // nobody asked for the choice at every row: draw only at the rows the walk stands on
        const cudaError_t el = launch_sampled_walk(target_logits, dt, row_stride_elems, R, B + 1, V, L, n_rows, c, row_uniform,
                                                   node_token, node_parent, accept_len, accept_nodes, accept_tokens, bonus_token, st);
        if (el != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept_sampled: walk kernel: %s", cudaGetErrorString(el));
        return DDTREE_OK;
    }
    cudaError_t e = launch_row_argmax(target_logits, dt, row_stride_elems, R, B + 1, V, n_rows, lay.a, workspace, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept_sampled: maximum pass: %s", cudaGetErrorString(e));
    e = launch_row_sample(target_logits, dt, row_stride_elems, R, B + 1, V, n_rows, c, row_uniform, lay, workspace, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept_sampled: sampling pass: %s", cudaGetErrorString(e));
    const int32_t* choice = reinterpret_cast<const int32_t*>(static_cast<const char*>(workspace) + lay.off_tok);
    e = launch_accept_walk(R, B + 1, L, lay.a, workspace, choice, node_token, node_parent, n_rows, accept_len, accept_nodes,
                           accept_tokens, bonus_token, node_choice, st);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept_sampled: walk kernel: %s", cudaGetErrorString(e));
    return DDTREE_OK;
}

int ddtree_rope_tree(void* q, void* k_tree, const int32_t* position_ids, const int32_t* n_rows, int dt, int R, int B,
                     int Hq, int Hkv, int d, float rope_theta, void* cuda_stream) {
    if (R < 1 || B < 1 || Hq < 1 || Hkv < 1) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_rope_tree: R, B, Hq, Hkv must be >= 1");
    if (B > kMaxB) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_rope_tree: B %d > %d", B, kMaxB);
    if (dt != DDTREE_F32 && dt != DDTREE_BF16) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_rope_tree: unknown dtype %d", dt);
    if (d < 2 || d > 256 || (d & 1)) return fail(DDTREE_ERR_UNSUPPORTED, "ddtree_rope_tree: head_dim %d must be even and in [2, 256]", d);
    if (!(rope_theta > 0.f) || !(rope_theta <= 3.0e38f))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_rope_tree: rope_theta must be positive and finite");
    if (!position_ids || !n_rows) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_rope_tree: position_ids or n_rows is NULL");
    if (!q && !k_tree) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_rope_tree: both q and k_tree are NULL");
    const cudaError_t e = launch_rope_tree(q, k_tree, position_ids, n_rows, dt, R, B + 1, Hq, Hkv, d,
                                           std::log2(static_cast<double>(rope_theta)), static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_rope_tree: %s", cudaGetErrorString(e));
    return DDTREE_OK;
}

int ddtree_kv_compact(int R, int B, int L, int Hkv, int d, int dt, int layers, const void* const* k_tree,
                      const void* const* v_tree, void* const* k_cache, void* const* v_cache, const int64_t* dst_row,
                      const int32_t* accept_len, const int32_t* accept_nodes, void* cuda_stream) {
    if (R < 1 || B < 1 || L < 1 || Hkv < 1 || d < 1 || layers < 1)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: R, B, L, Hkv, d, layers must be >= 1");
    if (B > kMaxB) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: B %d > %d", B, kMaxB);
    if (L > kMaxL) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: L %d > %d", L, kMaxL);
    if (dt != DDTREE_F32 && dt != DDTREE_BF16) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: unknown dtype %d", dt);
    const int64_t row_bytes = static_cast<int64_t>(Hkv) * d * elem_size(dt);
    if (row_bytes % 16 || row_bytes > (1 << 24))
        return fail(DDTREE_ERR_UNSUPPORTED, "ddtree_kv_compact: a K/V row (%lld bytes) must be a multiple of 16 bytes",
                    static_cast<long long>(row_bytes));
    if (!k_tree || !v_tree || !k_cache || !v_cache || !dst_row || !accept_len || !accept_nodes)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: a required pointer is NULL");
    for (int l = 0; l < layers; ++l) {
        if (!k_tree[l] || !v_tree[l] || !k_cache[l] || !v_cache[l])
            return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: layer %d has a NULL buffer", l);
        if (!aligned16(k_tree[l]) || !aligned16(v_tree[l]) || !aligned16(k_cache[l]) || !aligned16(v_cache[l]))
            return fail(DDTREE_ERR_INVALID_ARG, "ddtree_kv_compact: layer %d: buffers must be 16-byte aligned", l);
    }
    const cudaError_t e = launch_kv_compact(R, B + 1, L, static_cast<int>(row_bytes), layers, k_tree, v_tree, k_cache, v_cache,
                                            dst_row, accept_len, accept_nodes, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_kv_compact: %s", cudaGetErrorString(e));
    return DDTREE_OK;
}

static int fill_attn_args(const char* fn, AttnArgs& a, const void* q, const void* k_cache, const void* v_cache,
                          const int32_t* cu_prefix_host, const int32_t* cu_prefix, const void* k_tree,
                          const void* v_tree, const uint32_t* anc_mask, const int32_t* n_rows, void* out, float* lse,
                          int dt, int R, int B, int Hq, int Hkv, int d, float scale, bool need_ptrs) {
    if (R < 1 || B < 1 || Hq < 1 || Hkv < 1 || d < 1)
        return fail(DDTREE_ERR_INVALID_ARG, "%s: R, B, Hq, Hkv, d must be >= 1", fn);
    if (B > kMaxB) return fail(DDTREE_ERR_INVALID_ARG, "%s: B %d > %d", fn, B, kMaxB);
    if (dt != DDTREE_F32 && dt != DDTREE_BF16) return fail(DDTREE_ERR_INVALID_ARG, "%s: unknown dtype %d", fn, dt);
    if (Hq % Hkv) return fail(DDTREE_ERR_INVALID_ARG, "%s: Hq %d is not a multiple of Hkv %d", fn, Hq, Hkv);
    const int G = Hq / Hkv;
    if (G != 1 && G != 2 && G != 4 && G != 8 && G != 16)
        return fail(DDTREE_ERR_UNSUPPORTED, "%s: Hq/Hkv = %d not in {1,2,4,8,16}", fn, G);
    if (dt == DDTREE_BF16 && d != 128) return fail(DDTREE_ERR_UNSUPPORTED, "%s: bf16 needs head_dim 128 (got %d)", fn, d);
    if (dt == DDTREE_F32 && d != 64 && d != 128)
        return fail(DDTREE_ERR_UNSUPPORTED, "%s: fp32 needs head_dim 64 or 128 (got %d)", fn, d);
    if (!cu_prefix_host) return fail(DDTREE_ERR_INVALID_ARG, "%s: cu_prefix_host is NULL", fn);
    int max_p = 0;
    if (cu_prefix_host[0] != 0) return fail(DDTREE_ERR_INVALID_ARG, "%s: cu_prefix_host[0] must be 0", fn);
    for (int r = 0; r < R; ++r) {
        const int p = cu_prefix_host[r + 1] - cu_prefix_host[r];
        if (p < 0) return fail(DDTREE_ERR_INVALID_ARG, "%s: cu_prefix_host is not non-decreasing", fn);
        if (p > max_p) max_p = p;
    }
    if (need_ptrs) {
        if (!q || !k_tree || !v_tree || !anc_mask || !n_rows || !out || !cu_prefix)
            return fail(DDTREE_ERR_INVALID_ARG, "%s: a required pointer is NULL", fn);
        if (cu_prefix_host[R] > 0 && (!k_cache || !v_cache))
            return fail(DDTREE_ERR_INVALID_ARG, "%s: k_cache/v_cache is NULL with a non-empty prefix", fn);
        if (!aligned16(q) || !aligned16(k_cache) || !aligned16(v_cache) || !aligned16(k_tree) || !aligned16(v_tree) ||
            !aligned16(out))
            return fail(DDTREE_ERR_INVALID_ARG, "%s: tensors must be 16-byte aligned", fn);
    }
    a.q = q; a.k_cache = k_cache; a.v_cache = v_cache; a.k_tree = k_tree; a.v_tree = v_tree;
    a.cu_prefix = cu_prefix; a.anc_mask = anc_mask; a.n_rows = n_rows; a.out = out; a.lse = lse;
    a.R = R; a.B = B; a.N = B + 1; a.W = (B + 1 + 31) / 32; a.Hq = Hq; a.Hkv = Hkv; a.G = G; a.d = d;
    if (!(scale >= 0.f) || !(scale <= 3.0e38f)) return fail(DDTREE_ERR_INVALID_ARG, "%s: softmax_scale must be positive and finite (0 = 1/sqrt(d))", fn);
    a.scale = scale != 0.f ? scale : 1.0f / sqrtf(static_cast<float>(d));
    a.max_prefix = max_p;
    a.total_prefix = cu_prefix_host[R];
    return DDTREE_OK;
}

size_t ddtree_tree_attention_workspace_bytes(int R, int B, int Hq, int Hkv, int d, int dt,
                                             const int32_t* cu_prefix_host) {
    AttnArgs a;
    if (fill_attn_args("ddtree_tree_attention_workspace_bytes", a, nullptr, nullptr, nullptr, cu_prefix_host, nullptr,
                       nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, dt, R, B, Hq, Hkv, d, 0.f, false))
        return 0;
    if (dt == DDTREE_F32) return 256;  // the fp32 kernel needs no scratch; a token size keeps callers uniform
    return tree_attention_bf16_workspace(a, cu_prefix_host);
}

int ddtree_tree_attention_kernel_count(int R, int B, int Hq, int Hkv, int d, int dt, const int32_t* cu_prefix_host) {
    AttnArgs a;
    if (fill_attn_args("ddtree_tree_attention_kernel_count", a, nullptr, nullptr, nullptr, cu_prefix_host, nullptr,
                       nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, dt, R, B, Hq, Hkv, d, 0.f, false))
        return 0;
    return dt == DDTREE_F32 ? 1 : tree_attention_bf16_kernels(a);
}

int ddtree_tree_attention(const void* q, const void* k_cache, const void* v_cache, const int32_t* cu_prefix_host,
                          const int32_t* cu_prefix, const void* k_tree, const void* v_tree, const uint32_t* anc_mask,
                          const int32_t* n_rows, void* out, float* lse_or_null, int dt, int R, int B, int Hq, int Hkv,
                          int d, float softmax_scale, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    AttnArgs a;
    int rc = fill_attn_args("ddtree_tree_attention", a, q, k_cache, v_cache, cu_prefix_host, cu_prefix, k_tree, v_tree,
                            anc_mask, n_rows, out, lse_or_null, dt, R, B, Hq, Hkv, d, softmax_scale, true);
    if (rc) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    if (dt == DDTREE_F32) {
        cudaError_t e = launch_tree_attention_f32(a, st);
        if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_tree_attention: %s", cudaGetErrorString(e));
        return DDTREE_OK;
    }
    const size_t need = tree_attention_bf16_workspace(a, cu_prefix_host);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_tree_attention: workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < need)
        return fail(DDTREE_ERR_WORKSPACE, "ddtree_tree_attention: workspace %zu < required %zu bytes", workspace_bytes, need);
    return launch_tree_attention_bf16(a, cu_prefix_host, workspace, workspace_bytes, st);
}

int ddtree_tree_attention_rope(const void* q, const void* k_cache, const void* v_cache, const int32_t* cu_prefix_host,
                               const int32_t* cu_prefix, const void* k_tree, const void* v_tree, const uint32_t* anc_mask,
                               const int32_t* n_rows, const int32_t* position_ids, float rope_theta, void* out,
                               float* lse_or_null, int dt, int R, int B, int Hq, int Hkv, int d, float softmax_scale,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
    AttnArgs a;
    int rc = fill_attn_args("ddtree_tree_attention_rope", a, q, k_cache, v_cache, cu_prefix_host, cu_prefix, k_tree, v_tree,
                            anc_mask, n_rows, out, lse_or_null, dt, R, B, Hq, Hkv, d, softmax_scale, true);
    if (rc) return rc;
    if (dt != DDTREE_BF16)
        return fail(DDTREE_ERR_UNSUPPORTED, "ddtree_tree_attention_rope: bf16 only (rotate fp32 rows with ddtree_rope_tree)");
    if (!position_ids) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_tree_attention_rope: position_ids is NULL");
    if (!(rope_theta > 0.f) || !(rope_theta <= 3.0e38f))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_tree_attention_rope: rope_theta must be positive and finite");
    a.rope = 1;
    a.position_ids = position_ids;
    a.rope_log2_theta = std::log2(static_cast<double>(rope_theta));
    const size_t need = tree_attention_bf16_workspace(a, cu_prefix_host);
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 15u))
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_tree_attention_rope: workspace is NULL or not 16-byte aligned");
    if (workspace_bytes < need)
        return fail(DDTREE_ERR_WORKSPACE, "ddtree_tree_attention_rope: workspace %zu < required %zu bytes", workspace_bytes, need);
    return launch_tree_attention_bf16(a, cu_prefix_host, workspace, workspace_bytes, static_cast<cudaStream_t>(cuda_stream));
}

// Scratch for ddtree_accept_static_scratch: lives in the library image, one copy per GPU that
// loads it.  Host code must not pass `g_static_scratch` itself to a kernel: in host code that name
// is only a handle for the runtime; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_scratch[DDTREE_STATIC_SCRATCH_BYTES];

// Device address of the scratch array on the current device (looked up once per device).
static int static_scratch_ptr(void** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static void* ptr[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_accept_static_scratch: cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices)
        return fail(DDTREE_ERR_UNSUPPORTED, "ddtree_accept_static_scratch: device index %d out of range", dev);
    std::lock_guard<std::mutex> g(mu);
    if (!ptr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_scratch);  // the current device is `dev`
        if (e != cudaSuccess || !p)
            return fail(DDTREE_ERR_CUDA, "ddtree_accept_static_scratch: cudaGetSymbolAddress: %s", cudaGetErrorString(e));
        ptr[dev] = p;
    }
    *out = ptr[dev];
    return DDTREE_OK;
}

int ddtree_accept_static_scratch(const void* target_logits, int dt, int64_t row_stride_elems, int R, int B, int V, int L,
                                 const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows,
                                 int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                                 int32_t* bonus_token, int32_t* node_argmax, void* cuda_stream) {
    if (R < 1 || B < 1 || B > kMaxB || V < 1)
        return fail(DDTREE_ERR_INVALID_ARG, "ddtree_accept_static_scratch: R, B, V out of range (got %d %d %d)", R, B, V);
    const size_t need = argmax_layout(R * (B + 1), V).total;
    if (need > DDTREE_STATIC_SCRATCH_BYTES)
        return fail(DDTREE_ERR_WORKSPACE,
                    "ddtree_accept_static_scratch: needs %zu bytes of scratch, the built-in array holds %u; "
                    "use ddtree_accept with a caller-provided workspace", need, DDTREE_STATIC_SCRATCH_BYTES);
    void* scratch = nullptr;
    const int rc = static_scratch_ptr(&scratch);
    if (rc) return rc;
    return ddtree_accept(target_logits, dt, row_stride_elems, R, B, V, L, node_token, node_parent, n_rows, accept_len,
                         accept_nodes, accept_tokens, bonus_token, node_argmax, scratch, DDTREE_STATIC_SCRATCH_BYTES,
                         cuda_stream);
}

int ddtree_tree_attention_set_path(int path) {
    if (path < 0 || path > 2) return fail(DDTREE_ERR_INVALID_ARG, "ddtree_tree_attention_set_path: path %d is not 0, 1 or 2", path);
    tree_attention_set_path(path);
    return DDTREE_OK;
}

int ddtree_selftest_wait_timeout(void* cuda_stream) {
    const cudaError_t e = launch_wait_timeout_selftest(4096u, static_cast<cudaStream_t>(cuda_stream));
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_selftest_wait_timeout: %s", cudaGetErrorString(e));
    return DDTREE_OK;
}

int ddtree_device_status(void) {
    uint32_t* p = device_status_word();
    if (!p) return fail(DDTREE_ERR_CUDA, "ddtree_device_status: no status word");
    cudaError_t e = cudaDeviceSynchronize();
    uint32_t v = 0;
    if (e == cudaSuccess) e = cudaMemcpy(&v, p, sizeof(v), cudaMemcpyDeviceToHost);
    if (e == cudaSuccess && v) e = cudaMemset(p, 0, sizeof(v));
    if (e != cudaSuccess) return fail(DDTREE_ERR_CUDA, "ddtree_device_status: %s", cudaGetErrorString(e));
    if (v) return fail(DDTREE_ERR_DEVICE_TIMEOUT, "a bounded device-side wait gave up (code 0x%x)", v);
    return DDTREE_OK;
}

}  // extern "C"

/*
 * ddtree.h -- C ABI of the DDTree per-round hot path for NVIDIA B200 (sm_100a).
 *
 * One speculative-decoding round of DDTree (paper Section 4.1, steps 2-4) between the
 * drafter's logits and the next bonus token:
 *
 *   ddtree_build           step 2 + the "compile" half of step 3: per-position log-softmax and
 *                          top-K (Sections 3 and 4.3), best-first selection of at most B prefixes
 *                          (Algorithm 1), flattening into verifier inputs (Section 4.4).
 *   ddtree_tree_attention  the attention of step 3: every tree row attends to the KV-cache prefix
 *                          and, inside the tree, to the root, its ancestors and itself (Section 4.4).
 *   ddtree_accept          step 4: greedy target choice at every row and the verifier walk
 *                          (Section 4.4, Figure 2(b)).
 *
 * Conventions
 *   - Every pointer is a DEVICE pointer unless its name ends in _host.  The caller owns every
 *     buffer, including the workspace; the library allocates no device memory in these calls and
 *     keeps no per-call state.  Buffers of one call must not overlap.
 *   - Every call validates its arguments on the host, ENQUEUES kernels on `cuda_stream`
 *     (a cudaStream_t; NULL = the legacy default stream) and returns.  Outputs are valid once
 *     the stream has been synchronised.  Nothing is launched when a call returns an error.
 *   - Return value: DDTREE_OK (0) or a positive ddtree_status.  ddtree_last_error() gives a
 *     thread-local message for the last failing call on the calling thread.
 *   - Conditions found on the device are data, not errors: when Algorithm 1's heap runs empty
 *     before B pops, n_rows < B+1 and the remaining rows are padding.
 *   - Shapes: R requests; L draft positions; V vocabulary; K tokens kept per position; B node
 *     budget (the root -- the bonus token b -- is not counted, Section 4.2), so a request has
 *     at most N = B+1 rows, row 0 being the root; W = ceil(N/32) mask words per row.
 *   - Limits: 1 <= K <= 32, K <= V, 1 <= L <= 32, 1 <= B <= 1024 (the largest budget the paper
 *     uses, Appendix B), V < 2^31.  Logits must be finite (the paper assumes q_i(v) in (0,1)).
 *   - Rows of logits must start on 16-byte boundaries (base pointer and row stride); V itself
 *     may be any size, a ragged tail is read element-wise.
 *   - Calls are re-entrant; the only hidden state is a per-process cache of device properties
 *     and TMA descriptors behind a mutex.
 */
#ifndef DDTREE_H_
#define DDTREE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    DDTREE_OK = 0,
    DDTREE_ERR_INVALID_ARG = 1, /* null required pointer, size out of range, misaligned rows    */
    DDTREE_ERR_UNSUPPORTED = 2, /* valid request this build has no kernel for (e.g. head_dim)   */
    DDTREE_ERR_WORKSPACE = 3,   /* workspace smaller than the *_workspace_bytes() answer         */
    DDTREE_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed; see ddtree_last_error()    */
    DDTREE_ERR_DEVICE_TIMEOUT = 5 /* a bounded device-side wait gave up (read via ddtree_device_status) */
} ddtree_status;

typedef enum { DDTREE_F32 = 0, DDTREE_BF16 = 1 } ddtree_dtype;

/* Static, never-freed strings. */
const char* ddtree_status_string(int status);
const char* ddtree_last_error(void);

/* ------------------------------------------------------------------------------------------
 * ddtree_build -- Sections 3, 4.3 (Algorithm 1) and 4.4 (the verifier's inputs: the tree as one
 * sequence, position ids, the attention mask).
 *
 * For every request r and draft position i = 1..L, reads the logit row l_i (row r*L + i-1 of
 * `drafter_logits`, V elements of type `dt`, rows `row_stride_elems` apart), forms
 * log q_i = l_i - logsumexp(l_i) in fp32 and keeps the K most probable tokens ordered by
 * (logit descending, token id ascending).  It then runs Algorithm 1: a max-heap keyed by
 * sigma(rho) = sum_i log q_i^(rho_i), started at the tuple (1); each pop adds a node and pushes
 * its next sibling (rank <= K) and first child (depth < L); it stops after B pops or when the
 * heap is empty.  The selected prefixes are written in LEVEL ORDER -- sorted by (depth, rank
 * tuple) -- so that row 0 is the root, parents precede children and siblings are adjacent in
 * rank order; this order depends only on the node set, not on the pop order.
 *
 * Inputs
 *   drafter_logits  [R*L rows, V]  dt = F32 or BF16
 *   root_token      [R] int32      bonus token b carried into the round (Section 3)
 *   prefix_len      [R] int32      tokens already in the KV cache; b sits at this position
 * Outputs (all [R, B+1] int32 unless noted; rows >= n_rows[r] are padding)
 *   n_rows          [R]            1 + number of selected nodes
 *   node_token                     token id per row (row 0 = root_token); padding -1
 *   node_parent                    parent row (row 0 = -1); padding -1
 *   node_depth                     depth (row 0 = 0); padding -1
 *   position_ids                   prefix_len + depth; padding -1
 *   anc_mask        [R, B+1, W] uint32  bit j of row i set iff row j is i itself or an ancestor
 *                                  of i (bit j lives in word j/32, bit j%32); padding rows 0
 *   first_child, child_count       optional (NULL to skip): first child row (-1 if none), #children
 *   node_logprob    [R, B+1] fp32  optional: sigma of the row's prefix (root 0, padding 0).  fp32
 *                                  arithmetic: compare with a tolerance, never bit-for-bit
 *   topk_token      [R, L, K] int32, topk_logprob [R, L, K] fp32   optional: the per-position table
 *   workspace                      at least ddtree_build_workspace_bytes(...) bytes, 16-byte aligned
 * ------------------------------------------------------------------------------------------ */
size_t ddtree_build_workspace_bytes(int R, int L, int V, int K, int B);

int ddtree_build(const void* drafter_logits, int dt, int64_t row_stride_elems,
                 int R, int L, int V, int K, int B,
                 const int32_t* root_token, const int32_t* prefix_len,
                 int32_t* n_rows, int32_t* node_token, int32_t* node_parent, int32_t* node_depth,
                 int32_t* position_ids, uint32_t* anc_mask,
                 int32_t* first_child, int32_t* child_count, float* node_logprob,
                 int32_t* topk_token, float* topk_logprob,
                 void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_tree_attention -- Section 4.4 (tree attention), Appendix B (scaled-dot-product
 * attention with an explicit tree mask is what the paper runs).
 *
 * For request r, row i < n_rows[r] and query head h (KV head h / (Hq/Hkv)):
 *   keys/values = the request's P_r cached rows (all visible) followed by the tree rows j whose
 *   bit is set in anc_mask[r, i];  out = softmax(q . k * softmax_scale) @ v.
 * The cache is packed: request r owns rows cu_prefix[r] .. cu_prefix[r+1]-1.
 *
 * Inputs
 *   q                [R, B+1, Hq, d]
 *   k_cache, v_cache [sum P, Hkv, d]      d contiguous
 *   cu_prefix_host   [R+1] int32 HOST     exclusive prefix sums of the P_r (used for planning: KV splits,
 *                                         workspace size, longest-first dispatch of the requests)
 *   cu_prefix        [R+1] int32 device   the same values on the device
 *   k_tree, v_tree   [R, B+1, Hkv, d]     this round's K/V of the tree rows (not yet in the cache)
 *   anc_mask         [R, B+1, W] uint32, n_rows [R] int32   as written by ddtree_build
 * Outputs
 *   out              [R, B+1, Hq, d]      same element type as q; rows >= n_rows[r] are left untouched
 *   lse_or_null      [R, B+1, Hq] fp32    optional natural-log sum of exp(scaled scores)
 * dt = DDTREE_BF16: bf16 inputs, fp32 accumulation on the tensor cores, probabilities rounded to
 *   bf16 before the PV product; requires d == 128.  When the KV range of a request is split over
 *   several CTAs (batches that do not fill the GPU), each part's normalised rows pass through fp16 before
 *   they are merged: the values must then stay below fp16's largest finite value, |v| < 65504 (an output
 *   row is a convex combination of V rows).  dt = DDTREE_F32: fp32 FMA arithmetic; d in {64, 128}.
 *   Hq must be a multiple of Hkv with Hq/Hkv in {1, 2, 4, 8, 16}.
 * Rows the call must ignore may hold anything, NaN and Inf bit patterns included: rows >= n_rows[r] of q,
 *   k_tree and v_tree, and memory behind the packed cache.  (A masked key's probability is zero, but its
 *   value row still travels through the tensor cores in a 128-key tile; the kernel clears such rows first.)
 *   Visible keys and values must be finite.
 * softmax_scale 0 means 1/sqrt(d); it must be positive.  All tensors must be 16-byte aligned.
 * workspace: at least ddtree_tree_attention_workspace_bytes(...) bytes, 16-byte aligned.
 * ------------------------------------------------------------------------------------------ */
size_t ddtree_tree_attention_workspace_bytes(int R, int B, int Hq, int Hkv, int d, int dt,
                                             const int32_t* cu_prefix_host);

int ddtree_tree_attention(const void* q, const void* k_cache, const void* v_cache,
                          const int32_t* cu_prefix_host, const int32_t* cu_prefix,
                          const void* k_tree, const void* v_tree,
                          const uint32_t* anc_mask, const int32_t* n_rows,
                          void* out, float* lse_or_null,
                          int dt, int R, int B, int Hq, int Hkv, int d, float softmax_scale,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_accept -- Section 4.4, Figure 2(b) (verifier walk under the greedy decoding rule).
 *
 * node_argmax[r, i] = smallest token id attaining the maximum of target logit row r*(B+1)+i.
 * Walk: cur = 0; while some child c of cur has node_token[c] == node_argmax[cur]: accept c,
 * cur = c.  bonus_token = node_argmax[cur] (the first unmatched target token, next round's root).
 *
 * Inputs
 *   target_logits [R*(B+1) rows, V]   dt = F32 or BF16; rows >= n_rows[r] are never read
 *   node_token, node_parent [R, B+1], n_rows [R]   as written by ddtree_build (any order with
 *                                     parent row < child row is accepted)
 * Outputs
 *   accept_len    [R]      number of accepted DRAFTED nodes, 0..L (the bonus token is not counted;
 *                          tokens committed this round = accept_len + 1)
 *   accept_nodes  [R, L]   rows of the accepted path in order, -1 padded
 *   accept_tokens [R, L]   their tokens, -1 padded
 *   bonus_token   [R]
 *   node_argmax   [R, B+1] optional; padding rows -1
 * ------------------------------------------------------------------------------------------ */
size_t ddtree_accept_workspace_bytes(int R, int B, int V);

int ddtree_accept(const void* target_logits, int dt, int64_t row_stride_elems,
                  int R, int B, int V, int L,
                  const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows,
                  int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                  int32_t* bonus_token, int32_t* node_argmax,
                  void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_accept_sampled -- Section 4.4 (verifier walk when the target decodes by sampling at a
 * temperature instead of greedily; the paper lets the verification use either rule).  The walk is that of
 * ddtree_accept; the target's choice at a row is a draw from softmax(target_logits[row] / temperature)
 * instead of the arg-max.
 *
 * The paper does not say how the draw is made.  Here it is a function of the row, the temperature and
 * one caller-supplied 32-bit integer per row, defined on integers so that it does not depend on the
 * order in which anything is summed:
 *   c    = (float)(log2(e) / (double)temperature)
 *   W_v  = floor(2^40 * e_v),  e_v = 2^((x_v - max_v x_v) * c) evaluated in float32 with one rounding per
 *          operation: t = (x_v - max) * c;  W_v = 0 if not t >= -40;  r = t + 12582912.0f (1.5 * 2^23: r is t
 *          rounded to the nearest integer, ties to even, plus that constant);  n = (int)bits(r) - 0x4B400000;
 *          f = t - (r - 12582912.0f), in [-1/2, 1/2];
 *          p = ((((a5 f + a4) f + a3) f + a2) f + a1) f + 1  (multiply, round, add, round; a1..a5 =
 *          0.693147004f, 0.240222424f, 0.0555073358f, 0.00967151299f, 0.00132647273f; |p / 2^f - 1| < 2e-7);
 *          with p = sig * 2^(e - 23) (sig its 24-bit significand, e in {-1, 0}) and sh = e + 17 + n:
 *          W_v = sig << sh if sh >= 0, else sig >> -sh   (the maximum gets exactly 2^40)
 *   choice = smallest v with W_0 + ... + W_v > floor((sum_v W_v) * k / 2^32),  k = row_uniform[row]
 * i.e. an inverse-CDF draw in token order with u = k / 2^32.  Supplying independent uniform k per row
 * makes every visited row's choice an independent draw; a row's draw does not depend on the others.
 *
 * Inputs as for ddtree_accept, plus
 *   temperature                      > 0 (a float: the value is used as passed)
 *   row_uniform   [R, B+1] uint32    device memory; entries of padding rows are not read
 * Outputs as for ddtree_accept; node_choice [R, B+1] (optional) receives the drawn token of every row,
 * padding rows -1.  A row whose logits have no finite maximum gets choice -1 (the walk stops there).
 * The walk only consults the rows it stands on (the root and the accepted nodes: at most L + 1 per
 * request).  With node_choice == NULL the call draws at those rows only: one cluster of CTAs per request
 * follows the walk and reads each visited row once (vocabularies up to 458,000 tokens; larger ones, and
 * calls that ask for node_choice, weigh every row in passes over all target logits).  The draw, and so every
 * output, is the same either way.
 * V <= 2^22.  Errors as for ddtree_accept; temperature <= 0 or not finite -> DDTREE_ERR_INVALID_ARG.
 * ------------------------------------------------------------------------------------------ */
size_t ddtree_accept_sampled_workspace_bytes(int R, int B, int V);

int ddtree_accept_sampled(const void* target_logits, int dt, int64_t row_stride_elems,
                          int R, int B, int V, int L,
                          const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows,
                          float temperature, const uint32_t* row_uniform,
                          int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                          int32_t* bonus_token, int32_t* node_choice,
                          void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_rope_tree -- Section 4.4 (position ids follow the tree depth, so that the verifier encodes every
 * node at the position it would have in its own branch).  Applies the rotary positional encoding (half-split
 * form, as the paper's Qwen3 targets use) to the tree's query and key rows IN PLACE, at the position ids
 * ddtree_build wrote:
 * for every valid row i, every head and every j < d/2, with a = position_ids[r, i] * rope_theta^(-2j/d),
 *     (x[j], x[j + d/2])  <-  (x[j] cos a - x[j + d/2] sin a,  x[j + d/2] cos a + x[j] sin a).
 * Angles are evaluated in double precision, the rotation in float32, results rounded to dt.
 * Call it on a layer's q and k_tree before ddtree_tree_attention (the cached keys were rotated when they
 * were produced).  A pass of its own rather than a step inside the attention kernel: there every K row would
 * be rotated again by each CTA that loads it.
 *
 *   q        [R, B+1, Hq, d]  or NULL      k_tree  [R, B+1, Hkv, d]  or NULL   (not both NULL), dt = F32 or BF16
 *   position_ids [R, B+1], n_rows [R]      as written by ddtree_build; rows >= n_rows[r] are left untouched
 *   d even, 2..256; rope_theta > 0 (10^6 for Qwen3)
 * Errors: DDTREE_ERR_INVALID_ARG / DDTREE_ERR_UNSUPPORTED before anything is launched.
 * ------------------------------------------------------------------------------------------ */
int ddtree_rope_tree(void* q, void* k_tree, const int32_t* position_ids, const int32_t* n_rows,
                     int dt, int R, int B, int Hq, int Hkv, int d, float rope_theta, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_tree_attention_rope -- ddtree_tree_attention with the rotary positional encoding of Section 4.4
 * (position ids by tree depth) applied inside the kernel's load path: q and k_tree are given UNROTATED and are
 * not modified; every CTA rotates its query tile in shared memory once, before its first product, and the
 * tiles of tree keys as they are staged (the cached keys were rotated when they were produced and are used as
 * they are).  Same rule as ddtree_rope_tree: pair (j, j + d/2) of every head of row i is rotated by
 * position_ids[r, i] * rope_theta^(-2j/d); angles in double precision, rotation in float32, rotated values
 * rounded to bf16 before the products (as a separate ddtree_rope_tree pass would store them).  Equivalent to
 * ddtree_rope_tree on copies of q and k_tree followed by ddtree_tree_attention.
 *
 * Arguments as for ddtree_tree_attention, plus position_ids [R, B+1] (as written by ddtree_build; a row sits
 * at most 32 positions behind row 0 of its request) and rope_theta > 0.  dt must be DDTREE_BF16 (d = 128).
 * The workspace size is ddtree_tree_attention_workspace_bytes(...).
 * ------------------------------------------------------------------------------------------ */
int ddtree_tree_attention_rope(const void* q, const void* k_cache, const void* v_cache,
                               const int32_t* cu_prefix_host, const int32_t* cu_prefix,
                               const void* k_tree, const void* v_tree,
                               const uint32_t* anc_mask, const int32_t* n_rows,
                               const int32_t* position_ids, float rope_theta,
                               void* out, float* lse_or_null,
                               int dt, int R, int B, int Hq, int Hkv, int d, float softmax_scale,
                               void* workspace, size_t workspace_bytes, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_accept_static_scratch -- the paper has no counterpart; this is a packaging variant of
 * ddtree_accept for callers that cannot hand over a workspace.
 *
 * Who needs it: code that runs where device memory can no longer be obtained -- a decoding loop
 * inside a serving engine whose memory pool was carved up at start-up (every byte belongs to the
 * KV cache or to activations, and cudaMalloc at this point would either fail or stall every
 * stream of the process while the driver maps memory), a plug-in that is handed tensors but has
 * no allocator of its own, or a real-time thread that must not enter the driver's allocation
 * path.  Such a caller still owns its inputs and outputs; what it lacks is a place for the
 * per-chunk (max, arg-max) partials of the target-logits pass.
 *
 * Same arguments, outputs and errors as ddtree_accept without the workspace pair.  The partials
 * go to a fixed array inside the library (DDTREE_STATIC_SCRATCH_BYTES bytes of device memory per
 * GPU, held from the moment the library is loaded on that GPU until the process exits).
 *   - Limit: ddtree_accept_workspace_bytes(R, B, V) must not exceed DDTREE_STATIC_SCRATCH_BYTES;
 *     larger problems are refused with DDTREE_ERR_WORKSPACE and nothing is launched.
 *   - The first call on each device looks up the array's device address (one driver query, no
 *     allocation).  Make that first call outside any stream capture.
 *   - Every call on a device uses the same array.  Nothing in it has to start at zero (every
 *     partial that is read was written by the same call), but two calls whose kernels overlap on
 *     the GPU -- different streams, or different host threads -- overwrite each other's partials:
 *     serialise them (one stream, or an event between them).
 *   - The call itself allocates nothing, neither on the device nor through any library.
 * ------------------------------------------------------------------------------------------ */
#define DDTREE_STATIC_SCRATCH_BYTES (256u * 1024u)

int ddtree_accept_static_scratch(const void* target_logits, int dt, int64_t row_stride_elems,
                                 int R, int B, int V, int L,
                                 const int32_t* node_token, const int32_t* node_parent, const int32_t* n_rows,
                                 int32_t* accept_len, int32_t* accept_nodes, int32_t* accept_tokens,
                                 int32_t* bonus_token, int32_t* node_argmax, void* cuda_stream);

/* ------------------------------------------------------------------------------------------
 * ddtree_kv_compact -- Section 4.4, end of a round: after the walk only the accepted path stays
 * in the KV cache.  For every layer l and request r the rows of the root (tree row 0) and of the
 * accept_len[r] accepted nodes are copied, in path order, from this round's tree buffers to the
 * cache rows dst_row[r], dst_row[r] + 1, ..., so that every token sits at the position id it was
 * verified at (prefix_len + depth).  Nothing else in the cache is touched.  Pure data movement,
 * all layers in one launch (one more per 64 layers).
 *
 *   k_tree, v_tree   HOST arrays of `layers` DEVICE pointers, each [R, B+1, Hkv, d] (dt)
 *   k_cache, v_cache HOST arrays of `layers` DEVICE pointers, each [rows, Hkv, d] (dt); the caller
 *                    guarantees rows > dst_row[r] + accept_len[r] for every r (one launch cannot
 *                    check capacities it is not told)
 *   dst_row          DEVICE [R] int64: cache row that receives the root of request r; for the packed
 *                    layout of ddtree_tree_attention this is cu_prefix[r] + prefix_len[r], which
 *                    needs spare rows behind each request's prefix (trivially so for R = 1)
 *   accept_len, accept_nodes   DEVICE, as written by ddtree_accept ([R] and [R, L])
 * Hkv * d * sizeof(dt) must be a multiple of 16 bytes and all buffers 16-byte aligned.  The pointer
 * arrays are read during the call only.  Errors: as for the other entry points; nothing is
 * launched when an argument is refused.
 * ------------------------------------------------------------------------------------------ */
int ddtree_kv_compact(int R, int B, int L, int Hkv, int d, int dt, int layers,
                      const void* const* k_tree, const void* const* v_tree,
                      void* const* k_cache, void* const* v_cache, const int64_t* dst_row,
                      const int32_t* accept_len, const int32_t* accept_nodes, void* cuda_stream);

/* Device-side status word of the current device: 0, or DDTREE_ERR_DEVICE_TIMEOUT if a bounded
 * wait inside a kernel of this library gave up since the last call.  Synchronises the device,
 * reads and clears the word. */
int ddtree_device_status(void);

/* Self-test of that reporting path (no counterpart in the paper).  Every wait inside the attention
 * kernel (on a TMA copy, on the tensor pipe, on another warp) polls a bounded number of times; when
 * the bound runs out the kernel raises the time-out flag in the status word, waits for its own
 * copies in flight, frees its tensor memory and returns: the context stays usable and no output is
 * trusted.  This call enqueues a one-thread kernel with such a wait on a barrier that nothing ever
 * arrives at and a bound of a few thousand polls (microseconds), so that after it
 * ddtree_device_status() returns DDTREE_ERR_DEVICE_TIMEOUT once and DDTREE_OK afterwards.  The
 * kernel does not trap, fault or spin without bound. */
int ddtree_selftest_wait_timeout(void* cuda_stream);

/* Which bf16 attention kernel ddtree_tree_attention launches (no counterpart in the paper; a tuning and
 * test hook).  The library has two: one whose CTAs hold two 128-row tiles of a KV head (the throughput
 * kernel: batches that fill the SMs, long KV ranges) and one whose CTAs hold a single row tile with two
 * threads per row (the latency kernel: a batch whose row tiles leave SMs idle unless the KV range is cut
 * into a few tiles per CTA).  path 0 (the default) lets a cost model choose per call from the shapes; 1
 * forces the first, 2 the second wherever it applies (all CTAs resident at once, no rotary variant).
 * Process-wide, takes effect at the next call; the workspace size ddtree_tree_attention_workspace_bytes
 * reports covers every choice.  Both kernels give results within the same tolerance of each other, not
 * bit-identical ones.  Returns DDTREE_OK, or DDTREE_ERR_INVALID_ARG for a path outside 0..2. */
int ddtree_tree_attention_set_path(int path);

/* How many kernels of this library one ddtree_tree_attention call with these shapes launches under the current
 * path setting: 1, or 2 when the KV range is split and a merge kernel follows (no counterpart in the paper; for
 * launch accounting in benchmarks).  Arguments as for ddtree_tree_attention_workspace_bytes; 0 if they are invalid. */
int ddtree_tree_attention_kernel_count(int R, int B, int Hq, int Hkv, int d, int dt, const int32_t* cu_prefix_host);

#ifdef __cplusplus
}
#endif
#endif /* DDTREE_H_ */

/*
 * wide.h -- C ABI of the WIDE hot path for NVIDIA B200 (sm_100a).
 *
 * Token-wise dynamic-width execution of a transformer layer:
 *   wide_route      router scores -> per-token group bitmask      (Section 3.1, Eq. 4)
 *   wide_reorder    per-group mask reordering + tile predicates   (Section 3.3, Eq. 6-8, Algorithm 1)
 *   wide_ffn        block-skipping SwiGLU FFN                     (Eq. 3; Algorithms 2 and 3)
 *   wide_oproj      head-group-masked attention output projection (Eq. 2; Eq. 10, Algorithm 3)
 *   wide_attn       head-group-masked causal attention            (Eq. 1; Algorithm 4: prefill and decode forms)
 *   wide_qproj      routed query projection, GEMM-MN              (Eq. 1 under the mask; Algorithm 2)
 *   wide_unpermute  the scatter epilogue as a standalone step     (Algorithm 2, epilogue)
 *
 * General rules
 *   - Every data pointer is a DEVICE pointer owned by the caller; the library never
 *     allocates, frees or keeps caller-visible memory.  Scratch memory is passed in as
 *     `workspace` (size from wide_workspace_bytes); a few small buffers (decode accumulators,
 *     completion counters, the partial results of the decode attention) belong to the context
 *     and are allocated once by wide_create, which is why one context must not run two calls
 *     concurrently on different streams.
 *   - All work is enqueued on the caller's stream (`stream` is a cudaStream_t cast to
 *     void*); no call synchronises the host or reads results back, except wide_status.
 *   - Matrices are row-major and contiguous.  Base pointers must be 16-byte aligned.
 *     Weights use the Linear layout C = A B^T with B in [N, K]:
 *       w_gate, w_up [d_ff, hidden]   w_down [hidden, d_ff]   w_o [hidden, attn_dim]
 *       w_router [n_groups, hidden]
 *   - Masks are bit-packed: bit (g % 32) of word mask_bits[t * W + g / 32], W = ceil(n_groups/32),
 *     is 1 iff token t executes group g; unused high bits are 0.
 *   - Return value: WIDE_OK or a negative WIDE_ERR_* code.  Argument errors are found on the
 *     host before anything is launched and leave all outputs untouched.
 *   - Outputs are fully overwritten (no accumulate-into semantics).
 *   - Device-side waits are bounded; if one expires the kernel records WIDE_ERR_TIMEOUT in
 *     the context's device status word and returns (it never traps or spins forever).
 */
#ifndef WIDE_H_
#define WIDE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define WIDE_VERSION 112

#if defined(__GNUC__)
#define WIDE_API __attribute__((visibility("default")))
#else
#define WIDE_API
#endif

/* error codes */
#define WIDE_OK 0
#define WIDE_ERR_INVALID_ARG (-1)
#define WIDE_ERR_UNSUPPORTED_SHAPE (-2)
#define WIDE_ERR_ALIGNMENT (-3)
#define WIDE_ERR_WORKSPACE (-4)
#define WIDE_ERR_CUDA (-5)
#define WIDE_ERR_TIMEOUT (-6)

/* element types of activations / weights / outputs */
#define WIDE_BF16 0
#define WIDE_F32 1

/* router forms */
#define WIDE_ROUTE_TOPK 0        /* one linear layer hidden -> n_groups, k largest per token   */
#define WIDE_ROUTE_PAIR_ARGMAX 1 /* bottleneck W1 W2 -> 2 logits per group, Eq. 4 (inference)  */

/* operations, for wide_workspace_bytes */
#define WIDE_OP_ROUTE 0
#define WIDE_OP_REORDER 1
#define WIDE_OP_FFN 2
#define WIDE_OP_OPROJ 3
#define WIDE_OP_UNPERMUTE 4

/* flags for wide_ffn / wide_oproj / wide_route */
#define WIDE_FLAG_NONE 0u
#define WIDE_FLAG_SIMT 1u        /* use the plain CUDA-core kernels (any shape; the only path for fp32) */
#define WIDE_FLAG_FORCE_PREFILL 2u /* tokens <= WIDE_DECODE_MAX_TOKENS would normally take the decode path */
#define WIDE_FLAG_FORCE_DECODE 4u  /* take the union-streaming decode path (tokens <= WIDE_DECODE_MAX_TOKENS) */
#define WIDE_FLAG_INPUT_MASKED 8u  /* wide_oproj: attn_out already holds exact zeros for every inactive
                                      (token, group) pair, as wide_attn writes it; the prefill path then
                                      skips its masking pass (and the token clustering that rides on it) */

#define WIDE_FLAG_KAXIS_GROUP 16u   /* wide_ffn / wide_oproj prefill: run the K-axis product in its per-group
                                      form (Algorithm 3: only the active (tile, group) blocks, partial sums
                                      reduced into the output), whatever the group size and active fraction */
#define WIDE_FLAG_KAXIS_OWNER 32u   /* ... in its owner-computes form (a token tile walks all groups its
                                      tokens use; no reduction traffic).  Default: chosen on the device from
                                      the mask, see wide_oproj */
#define WIDE_FLAG_REDUCE_BF16 64u   /* per-group form with a bf16 output: add the partial sums (one per active
                                      group of a token) in bf16 straight into the output instead of in fp32
                                      scratch; halves the reduction traffic.  Default when n_groups <= 16 */
#define WIDE_FLAG_DECODE_TC 128u    /* decode path with at most WIDE_DECODE_GEMV_MAX_TOKENS tokens: take the
                                      tensor-core kernel instead of the matrix-vector kernel (the GEMV
                                      dispatch for tiny M of Appendix B), which is the default there */

#define WIDE_DECODE_MAX_TOKENS 64
#define WIDE_DECODE_GEMV_MAX_TOKENS 2
#define WIDE_MAX_GROUPS 256

typedef struct wide_ctx wide_ctx;

/* Create / destroy a context bound to CUDA device `device` (ordinal).  The context holds the
 * device properties, a few device status / barrier words and the fp32 accumulators of the decode
 * path (21 MB, kept zero between calls).  Host-synchronous.  A context serves one stream at a
 * time: calls issued through the same context must not overlap on the GPU. */
WIDE_API int wide_create(wide_ctx** ctx, int device);
WIDE_API int wide_destroy(wide_ctx* ctx);

/* Synchronise `stream`, read the device status word into *status (WIDE_OK or
 * WIDE_ERR_TIMEOUT) and clear it; after a timeout the context's internal buffers are reset.
 * The only call that blocks the host.
 * After a device-side wait has expired the context's counters and accumulators are in an
 * undefined state: until wide_status has been called, every decode-path call on the context
 * finds the status word set when its kernel starts and returns without touching its outputs. */
WIDE_API int wide_status(wide_ctx* ctx, void* stream, int* status);

/* Override the bound of every device-side wait (nanoseconds; default 2e9). */
WIDE_API int wide_set_wait_limit_ns(wide_ctx* ctx, uint64_t ns);

/* Self-test of the failure path (no counterpart in the paper): one CTA waits, with the context's
 * wait bound, on an mbarrier that is never completed; when the bound expires it sets the status
 * word as a hot-path kernel would and returns.  After that wide_status reports WIDE_ERR_TIMEOUT
 * and the context stays usable.  Nothing faults or hangs.  Errors: INVALID_ARG, CUDA. */
WIDE_API int wide_selftest_wait(wide_ctx* ctx, void* stream);

/* Per-kernel timing (tracing aid).  wide_profile_begin creates `max_records` CUDA event pairs;
 * until wide_profile_end every kernel the library launches is bracketed by one pair on its
 * stream.  wide_profile_end synchronises `stream` and writes one text line per kernel name,
 * "name,launches,total_ms\n", into buf (NUL-terminated), then frees the events.  Not for use
 * during stream capture.  wide_launch_count returns the number of kernels launched through this
 * context since it was created. */
WIDE_API int wide_profile_begin(wide_ctx* ctx, int max_records);
WIDE_API int wide_profile_end(wide_ctx* ctx, void* stream, char* buf, size_t buf_bytes);
WIDE_API int wide_launch_count(wide_ctx* ctx, unsigned long long* count);

WIDE_API const char* wide_strerror(int code);
WIDE_API int wide_version(void);

/* Bytes of scratch the given operation needs for these shapes (0 if none).
 *   tokens T, hidden D, inner = d_ff (FFN) or attn_dim (O-proj), group G, n_groups N_G.
 * The same size is valid for every flag combination of that operation. */
WIDE_API size_t wide_workspace_bytes(int op, int dtype, int tokens, int hidden, int inner, int group, int n_groups);

/*
 * wide_route -- Section 3.1 "Routing components" (Eq. 4) and the fixed-budget reading of
 * Appendix A ("each token selects R groups").
 *
 *   mode WIDE_ROUTE_TOPK:        s[t,g] = sum_i x[t,i] * w_router[g,i];  token t executes the
 *                                k_t groups with the largest score, equal scores -> lower g.
 *                                k_t = k_per_token[t] if k_per_token != NULL else k.
 *                                w2 must be NULL, rank 0.
 *   mode WIDE_ROUTE_PAIR_ARGMAX: l = (x W1) W2 with w_router = W1 [hidden, rank] and
 *                                w2 = W2 [rank, 2*n_groups]; token t executes group g iff
 *                                l[t,2g] >= l[t,2g+1] (class 0 = execute, first index wins ties).
 *
 * The selection equals the one taken on fp64 sums of the exact input products, so it does not
 * depend on summation order.  (bf16, TOPK, hidden % 64 == 0: scores come from the tensor cores in
 * fp32 and every group closer to the selection boundary than an error bound is re-scored exactly
 * in fp64.  The bound assumes that the tensor-core accumulator loses at most 2^-23 of the running
 * sum per accumulated element; the parity tests check the measured error against it.  With at
 * most WIDE_DECODE_MAX_TOKENS tokens the same is done in one launch on the CUDA cores, fp32 sums
 * of hidden / 32-long chains with the same kind of bound; WIDE_FLAG_FORCE_PREFILL takes the
 * tensor-core form there too.  Other cases, and WIDE_FLAG_SIMT, compute all scores in fp64.)
 *   x          [tokens, hidden]  dtype
 *   mask_bits  out uint32 [tokens, W]
 *   scores     out fp32 [tokens, n_groups] (TOPK) or [tokens, 2*n_groups] (PAIR), may be NULL
 * Errors: INVALID_ARG (null pointer, k outside [0, n_groups], bad mode/dtype),
 *         UNSUPPORTED_SHAPE (n_groups > WIDE_MAX_GROUPS, hidden % 8 != 0), ALIGNMENT, WORKSPACE.
 */
WIDE_API int wide_route(wide_ctx* ctx, void* stream, const void* x, int dtype, int tokens, int hidden,
               const void* w_router, const void* w2, int rank, int n_groups, int mode, int k,
               const int32_t* k_per_token, uint32_t* mask_bits, float* scores, void* workspace,
               size_t workspace_bytes, unsigned flags);

/*
 * wide_route_static -- (no counterpart in the paper; a deployment variant of wide_route.)
 * Same arguments, results and errors as wide_route, minus the workspace: the fp64 score buffer is
 * a fixed array inside the library's device image.  It exists for hosts that may not allocate
 * device memory where they route -- a serving process whose own pool owns the whole heap, a
 * plugin called under another framework's allocator lock, a deployment that forbids cudaMalloc
 * after start-up.  The call itself allocates nothing on host or device.
 *   - Limit: the scratch the call needs, about tokens * (16 * n_groups + 8 * max(rank, 1) + 2176)
 *     bytes plus 1 KiB (wide_workspace_bytes(WIDE_OP_ROUTE, ...) is an upper bound), must not
 *     exceed WIDE_ROUTE_STATIC_BYTES (2 MiB: e.g. 580 tokens x 86 groups, 330 x 256); larger problems
 *     return WIDE_ERR_WORKSPACE and launch nothing.  Every GPU on which the library is loaded
 *     holds those 2 MiB until the process exits.
 *   - The first call on a device looks up the array's device address; it must be made with
 *     ctx's device current (else WIDE_ERR_INVALID_ARG) and should come before any stream
 *     capture.  Later calls reuse the cached address.  The cache is written without a lock: host
 *     threads that make that first call on one device at the same time all store the same
 *     value, which is harmless.
 *   - All calls on a device share the one array.  Nothing in it needs clearing between calls
 *     (each call overwrites what it reads), but two calls that overlap on the GPU -- different
 *     streams, or different contexts of the same device -- race on it: serialise them.
 */
#define WIDE_ROUTE_STATIC_BYTES (2u << 20)
WIDE_API int wide_route_static(wide_ctx* ctx, void* stream, const void* x, int dtype, int tokens, int hidden,
                               const void* w_router, const void* w2, int rank, int n_groups, int mode, int k,
                               const int32_t* k_per_token, uint32_t* mask_bits, float* scores, unsigned flags);

/*
 * wide_route_pair_prepare / wide_route_pair_norm -- Eq. 4 (Section 3.1, routing components) with the
 * router reading the layer's input through its RMSNorm, the weight-only work done once.
 *
 *   xh[t,:] = x[t,:] / sqrt(mean_i x[t,i]^2 + eps) * norm_weight      (norm_weight NULL: no scaling)
 *   l = (xh W1) W2,  token t executes group g iff l[t,2g] >= l[t,2g+1]
 *
 * The caller passes the UN-normalised hidden state: 1 / rms is a positive factor of a whole row and
 * cannot change which logit of a pair is larger, so the decision is taken on (x * norm_weight) W1 W2
 * and the factor only scales the logits that are returned.  norm_weight is folded into W1 by
 * wide_route_pair_prepare, which also forms, once per weight set,
 *   - diag(norm_weight) W1, transposed, as a pair of bf16 matrices (value and rounding remainder:
 *     the tensor-core product then misses the exact one by 2^-18 of its size at most), and
 *   - d_g = diag(norm_weight) W1 (W2[:,2g] - W2[:,2g+1]) in fp64 for every group,
 * so that a call is three launches: the bottleneck product on the tensor cores (fp32), the logits
 * with an error bound per pair, and one exact fp64 dot product x . d_g for each pair the bound
 * cannot decide (an exact tie falls back to the definition in fp64).  The selection equals the
 * fp64 decision on the exact input products.
 *   x [tokens, hidden] bf16; w1 [hidden, rank], w2 [rank, 2*n_groups], norm_weight [hidden] bf16
 *   prepared: device buffer of wide_route_pair_prepared_bytes(hidden, rank, n_groups), written by
 *       prepare, read by every later call with the same weights and shapes
 *   scores out fp32 [tokens, 2*n_groups] or NULL: the logits of the normalised input
 *   workspace: wide_route_pair_norm_workspace_bytes(tokens, rank)
 * Needs hidden % 64 == 0, hidden <= 16384, rank % 8 == 0, rank <= 32, n_groups <= 192.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE, ALIGNMENT, WORKSPACE, CUDA.
 */
WIDE_API size_t wide_route_pair_prepared_bytes(int hidden, int rank, int n_groups);
WIDE_API size_t wide_route_pair_norm_workspace_bytes(int tokens, int rank);
WIDE_API int wide_route_pair_prepare(wide_ctx* ctx, void* stream, const void* w1, const void* w2, const void* norm_weight,
                                     int hidden, int rank, int n_groups, void* prepared, size_t prepared_bytes);
WIDE_API int wide_route_pair_norm(wide_ctx* ctx, void* stream, const void* x, int tokens, int hidden, const void* w1,
                                  const void* w2, int rank, int n_groups, const void* norm_weight, float eps,
                                  const void* prepared, uint32_t* mask_bits, float* scores, void* workspace,
                                  size_t workspace_bytes);

/*
 * wide_reorder -- mask reordering, Eq. 6 / Algorithm 1, and the level-0 predicate of Eq. 7-8.
 * For each group g the rows are sorted by mask value, descending and STABLE (active rows in
 * ascending token order, then inactive rows in ascending token order).
 *
 *   perm       out int32 [n_groups, tokens]   perm[g][j] = token at sorted position j
 *   counts     out int32 [n_groups]           active tokens of group g
 *   tile_map   out uint8 [n_tiles, n_groups]  1 iff sorted rows [m*tile_m, (m+1)*tile_m) of group g
 *                                             contain an active row; n_tiles = ceil(tokens/tile_m)
 *   work_list  out int32 [n_tiles*n_groups, 2] the active (tile, group) pairs, group-major with
 *                                             tiles ascending; unused tail entries are (-1,-1)
 *   n_work     out int32 [1]
 *   union_list out int32 [n_groups]           groups with >= 1 active token, ascending; tail = -1
 *   n_union    out int32 [1]
 *   offsets    out int32 [n_groups + 1]       offsets[g] = sum_{g'<g} ceil(counts[g']/tile_m)*tile_m
 *                                             (row offsets of the packed-sorted layout)
 *   token_order, token_rank  out int32 [tokens] each, or both NULL.  One token permutation that puts
 *       tokens with the same mask next to each other, so that token tiles taken in this order share
 *       their active groups: token_order = the tokens in a STABLE sort by key(t), token_rank its
 *       inverse (token_rank[token_order[p]] = p), with
 *           n_groups <= 32:  key(t) = mask word 0 of token t & 0xFF  (the decisions for groups 0..7:
 *                            a tile of the sorted order agrees on the leading ones)
 *           n_groups  > 32:  key(t) = h >> 24,  h = 0x811C9DC5;  for each mask word w of token t:
 *                            h = (h ^ w) * 0x01000193  (32-bit wrap-around)
 *       The prefill FFN / O-projection keep their intermediate rows in this
 *       order and walk token tiles in it; a (tile, group) block is skipped when no token of the tile
 *       selected the group.
 * tile_m must be a power of two >= 16.  Errors: INVALID_ARG, UNSUPPORTED_SHAPE.
 */
WIDE_API int wide_reorder(wide_ctx* ctx, void* stream, const uint32_t* mask_bits, int tokens, int n_groups,
                 int tile_m, int32_t* perm, int32_t* counts, uint8_t* tile_map, int32_t* work_list,
                 int32_t* n_work, int32_t* union_list, int32_t* n_union, int32_t* offsets,
                 int32_t* token_order, int32_t* token_rank);

/*
 * wide_mask_slice -- the columns [group_begin, group_end) of a routing mask as a mask of their own
 * (bit g - group_begin of the output row = bit g of the input row, unused high bits 0).
 *
 * This is the mask a rank needs when the groups are sharded over GPUs (tensor parallelism over the
 * pruned dimension): Eq. 10 writes the K-axis product as a sum over groups, so the rank that holds
 * the gate / up rows and the down (or output-projection) columns of groups [group_begin, group_end)
 * computes its part of y by calling wide_reorder, wide_ffn / wide_oproj on ITS weight shard
 * (d_ff = (group_end - group_begin) * group, contiguous) with the sliced mask and an fp32 output;
 * the parts of all ranks add up to the full result (one reduce-scatter or all-reduce, the
 * caller's).  Routing itself is replicated: every rank scores all groups.
 *   mask_bits [tokens, ceil(n_groups/32)], out_bits out [tokens, ceil((group_end-group_begin)/32)]
 * Errors: INVALID_ARG (null pointer, range outside [0, n_groups]), UNSUPPORTED_SHAPE.
 */
WIDE_API int wide_mask_slice(wide_ctx* ctx, void* stream, const uint32_t* mask_bits, int tokens, int n_groups,
                             int group_begin, int group_end, uint32_t* out_bits);

/*
 * wide_ffn -- Eq. 3:  y = ((silu(x Wg^T) * (x Wu^T)) (.)_G M) Wd^T.
 * Gate/up columns and down rows of inactive (token, group) pairs are skipped (block level) or
 * contribute exact zeros (inside an active tile).
 *
 *   x [tokens, hidden], w_gate/w_up [d_ff, hidden], w_down [hidden, d_ff]: dtype
 *   mask_bits [tokens, W], W = ceil((d_ff/group)/32)
 *   perm, counts: outputs of wide_reorder for this mask.  Needed by the prefill tensor-core path;
 *       may be NULL when tokens <= WIDE_DECODE_MAX_TOKENS (decode path: union of active groups, no
 *       reordering) or with WIDE_FLAG_SIMT.
 *   token_order, token_rank: the token clustering of wide_reorder, or both NULL (tokens are then
 *       tiled in their original order).  Only the prefill tensor-core path uses them; the result
 *       is the same either way, block skipping in the down projection is not.
 *   y  out [tokens, hidden] of out_dtype
 * Tensor-core paths need dtype bf16, hidden % 64 == 0, group in {64,128,256,512}; other shapes
 * need WIDE_FLAG_SIMT (hidden % 4 == 0, group % 4 == 0).  The decode path serves up to
 * WIDE_DECODE_GEMV_MAX_TOKENS tokens with matrix-vector products on the CUDA cores (each needed
 * weight byte read once by plain loads) and more with the tensor-core kernel; WIDE_FLAG_DECODE_TC
 * takes the latter for any token count.  Same shapes, same results within the tolerance.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE, ALIGNMENT, WORKSPACE, CUDA.
 */
WIDE_API int wide_ffn(wide_ctx* ctx, void* stream, const void* x, const void* w_gate, const void* w_up,
             const void* w_down, int dtype, int tokens, int hidden, int d_ff, int group,
             const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts,
             const int32_t* token_order, const int32_t* token_rank, void* y, int out_dtype,
             void* workspace, size_t workspace_bytes, unsigned flags);

/*
 * wide_ffn_tp -- the FFN part of one rank when the groups are sharded over GPUs, with the
 * reduce-scatter of the parts fused into the down projection (Eq. 10 summed over this rank's groups;
 * the sum over ranks is a reduce-scatter over token rows).  Prefill sizes, tensor-core path only.
 *
 * x, w_gate, w_up, w_down, mask_bits_local, perm, counts, token_order, token_rank: as for wide_ffn on
 * this rank's weight shard (d_ff_local = this rank's groups * group; the mask sliced with
 * wide_mask_slice and reordered with wide_reorder).
 *   y_shards   HOST array of `world` DEVICE pointers: y_shards[r] = the fp32 shard
 *              [rows_per_rank, hidden] of rank r, which owns token rows [r * rows_per_rank,
 *              (r+1) * rows_per_rank); peer-mapped memory of the other GPUs for r != this rank
 *              (read when the call is made, not kept).  world <= 8, world * rows_per_rank >= tokens.
 * The down projection's epilogue adds every row of this rank's part into the shard of the rank
 * that owns the row (red.global.add.f32 over peer memory: plain peer stores, no multicast, no TMA on
 * peer memory).  The caller synchronises the ranks twice: every shard must be ZERO before any
 * rank's call starts, and a shard is complete when the calls of ALL ranks have finished.  A token
 * tile none of whose tokens uses any of this rank's groups sends nothing.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE (anything the tensor-core prefill path of wide_ffn does not
 * take), ALIGNMENT, WORKSPACE (wide_workspace_bytes(WIDE_OP_FFN, ...) is enough), CUDA.
 */
WIDE_API int wide_ffn_tp(wide_ctx* ctx, void* stream, const void* x, const void* w_gate, const void* w_up,
                         const void* w_down, int dtype, int tokens, int hidden, int d_ff_local, int group,
                         const uint32_t* mask_bits_local, const int32_t* perm, const int32_t* counts,
                         const int32_t* token_order, const int32_t* token_rank, float* const* y_shards, int world,
                         int rows_per_rank, void* workspace, size_t workspace_bytes);

/*
 * wide_oproj -- Eq. 2 / Eq. 10:  y[t,:] = sum_{g : M[t,g]=1} a[t, gG:(g+1)G] Wo[:, gG:(g+1)G]^T,
 * a = attention output flattened head-major [tokens, attn_dim], group g = channels [gG, (g+1)G).
 *   perm, counts: outputs of wide_reorder for this mask, or both NULL.  The prefill path has two
 *       K-axis kernels.  Per-group (Algorithm 3): for every active (128-row tile of a group's sorted
 *       active rows, group) block, the block's partial product is reduced into y -- the FLOPs are
 *       the active ones, the price is tokens * k * hidden partial sums through the L2 reduction
 *       units.  Owner-computes: a token tile walks the groups any of its tokens uses -- no reduction
 *       traffic, but nothing is skipped when every token has a mask of its own.  With perm / counts
 *       given and group >= 256 (group >= 128 with WIDE_FLAG_REDUCE_BF16) the kernels choose between
 *       the two on the device from the padded active fraction (no host read-back: the kernel that
 *       is not chosen returns at once); without them, or with a smaller group, owner-computes runs.  WIDE_FLAG_KAXIS_GROUP /
 *       WIDE_FLAG_KAXIS_OWNER override the choice, for wide_ffn's down projection as well.
 *       The per-group kernel sums in fp32 (in y itself when out_dtype is fp32, else in scratch that
 *       is converted at the end), or in bf16 straight into y when n_groups <= 16 or with
 *       WIDE_FLAG_REDUCE_BF16.
 *   token_order, token_rank as for wide_ffn (owner-computes kernel only).
 *   WIDE_FLAG_INPUT_MASKED: see the flag.
 */
WIDE_API int wide_oproj(wide_ctx* ctx, void* stream, const void* attn_out, const void* w_o, int dtype,
               int tokens, int hidden, int attn_dim, int group, const uint32_t* mask_bits,
               const int32_t* perm, const int32_t* counts, const int32_t* token_order,
               const int32_t* token_rank, void* y, int out_dtype, void* workspace,
               size_t workspace_bytes, unsigned flags);

/*
 * wide_attn -- Eq. 1 under the head-group mask, Algorithm 4.  For every active pair (token t,
 * routing group g) and every query head h of g:
 *     o[t, h, :] = sum_j softmax_j(scale * q[t, h, :] . k[j, h_kv, :]) v[j, h_kv, :]
 * over the keys j <= t + (tokens_k - tokens_q) when causal != 0, over all keys otherwise;
 * h_kv = h / (n_q_heads / n_kv_heads), routing group g = h / heads_per_group.  Inactive pairs,
 * and queries that see no key, give exact zeros.  K and V are dense (every token has them).
 *
 *   q   [tokens_q, n_q_heads * head_dim]  bf16, head-major (one sequence; tokens are positions)
 *   k,v [tokens_k, n_kv_heads * head_dim] bf16
 *   mask_bits [tokens_q, W]: the attention mask, n_groups = n_q_heads / heads_per_group
 *       <= WIDE_MAX_GROUPS.  Read by the decode form only; may be NULL (prefill form then).
 *   perm [n_groups, tokens_q], counts [n_groups]: outputs of wide_reorder for that mask.  Read by
 *       the prefill form only; may be NULL when the decode form runs.
 *   scale: multiplies the logits (<= 0 selects 1/sqrt(head_dim))
 *   o   out [tokens_q, n_q_heads * head_dim] bf16, fully overwritten
 * Prefill form (tcgen05): query tiles gathered through perm.  Decode form (the last paragraph of
 * the paper's attention section: reordering bypassed, routing checked per block, online softmax
 * split over the keys): taken when mask_bits is given and tokens_q * (n_q_heads / n_kv_heads) <= 8;
 * K and V of a KV head none of whose query rows is active are not read; the decode form brings K and
 * V in by TMA (n_kv_heads <= 256; CUDA cores for one query row per KV head, warp-level tensor-core
 * instructions for two to eight), or by plain loads with WIDE_FLAG_SIMT.  WIDE_FLAG_FORCE_PREFILL /
 * WIDE_FLAG_FORCE_DECODE override the choice.
 * All device pointers, 16-byte aligned, owned by the caller; nothing is allocated; work is
 * enqueued on `stream`.  Needs dtype bf16, head_dim 64 or 128, n_q_heads % n_kv_heads == 0,
 * n_q_heads % heads_per_group == 0.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE, ALIGNMENT, CUDA; a bounded device wait that expires
 * sets the status word (WIDE_ERR_TIMEOUT from wide_status).
 */
WIDE_API int wide_attn(wide_ctx* ctx, void* stream, const void* q, const void* k, const void* v, int dtype,
              int tokens_q, int tokens_k, int n_q_heads, int n_kv_heads, int head_dim,
              int heads_per_group, const uint32_t* mask_bits, const int32_t* perm, const int32_t* counts,
              int causal, float scale, void* o, unsigned flags);

/*
 * wide_qproj -- the query projection under the head-group mask (Section 3.1: only the active head
 * groups of a token compute their queries), Algorithm 2 (GEMM-MN) with a plain store epilogue:
 *     y[t, gG:(g+1)G] = x[t, :] W[gG:(g+1)G, :]^T   if group g is active for token t, else 0.
 *   x [tokens, hidden], w [n_out, hidden] (Linear layout), y out [tokens, n_out]: bf16
 *   perm [n_groups, tokens], counts [n_groups]: outputs of wide_reorder for the mask,
 *       n_groups = n_out / group <= WIDE_MAX_GROUPS
 * Needs dtype bf16, hidden % 64 == 0, group in {128, 256, 512}.  y is fully overwritten.
 * Errors: INVALID_ARG, UNSUPPORTED_SHAPE, ALIGNMENT, CUDA; WIDE_ERR_TIMEOUT through wide_status.
 */
WIDE_API int wide_qproj(wide_ctx* ctx, void* stream, const void* x, const void* w, int dtype, int tokens,
               int hidden, int n_out, int group, const int32_t* perm, const int32_t* counts, void* y,
               unsigned flags);

/*
 * wide_unpermute -- scatter epilogue of Algorithm 2 as its own call: packed-sorted rows back to
 * the dense token-major layout.
 *   dst[perm[g][j], g*G:(g+1)*G] = src_packed[offsets[g] + j, 0:G]   for j < counts[g]
 *   every other element of dst = 0
 *   src_packed [offsets[n_groups], group], dst [tokens, n_groups*group]; elem_bytes in {2, 4};
 *   group*elem_bytes must be a multiple of 16.
 */
WIDE_API int wide_unpermute(wide_ctx* ctx, void* stream, const void* src_packed, const int32_t* perm,
                   const int32_t* counts, const int32_t* offsets, int tokens, int n_groups,
                   int group, int elem_bytes, void* dst);

#ifdef __cplusplus
}
#endif
#endif /* WIDE_H_ */

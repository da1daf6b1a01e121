/*
 * dc.h -- C ABI of libdepthc: merging runs of convolutions into one convolution and
 * running the merged network's layers on an NVIDIA B200 (sm_100a).
 *
 * Source of the operations: arXiv 2301.12187, "Efficient Latency-Aware CNN Depth
 * Compression via Two-Stage Dynamic Programming" -- Sec. 3 (merging two convolutions,
 * f_{theta2}(f_{theta1}(X)) = f_{theta2 (*) theta1}(X)), Eq. 1 (theta^_i is the merge
 * of the run s_{i-1}+1..s_i), Sec. 2 / Sec. 5.1 (BN fused into the preceding
 * convolution), App. E.1 (skip addition folded into a single merged convolution),
 * App. E.2 (all zero padding of a run moved to its first convolution).
 *
 * Conventions
 *   - Feature maps are NHWC, dense, row-major: x[n][h][w][c].  dtype DC_F32 (float) or
 *     DC_BF16 (bfloat16 storage, fp32 accumulation).
 *   - Kernels handed in are fp32 [c_out][c_in/groups][k][k]; groups is 1 (dense) or
 *     c_in == c_out (depthwise).  Square odd k, symmetric zero padding, dilation 1.
 *   - Forward: y[n,Y,X,o] = act( b[o] + sum_{i,u,v} W[o,i,u,v] * x[n, Y*s+u-p, X*s+v-p, i] ),
 *     zero outside the image, H_out = floor((H + 2p - k)/s) + 1  (cross-correlation).
 *   - Every tensor pointer is a DEVICE pointer aligned to 16 bytes unless the argument is
 *     documented as a host pointer.  Descriptor structs (dc_layer, dc_geom, ...) are HOST
 *     memory and are only read during the call.
 *   - Ownership: the caller owns every buffer, workspaces included.  The library never
 *     allocates or frees device memory.
 *   - Every call enqueues work on `stream` and returns without synchronising, except
 *     dc_workspace_status and the *_host entry points, which say so.
 *   - Errors: a dc_status is returned; argument and shape errors are detected on the host
 *     before anything is launched.  Device-side waits are bounded; a wait that runs out
 *     latches DC_ERR_TIMEOUT in the first word of the caller's workspace (read it with
 *     dc_workspace_status) and the kernel returns without hanging.
 */
#ifndef DC_H_
#define DC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct CUstream_st *dc_stream; /* a cudaStream_t; NULL is the legacy default stream */

typedef enum {
  DC_OK = 0,
  DC_ERR_INVALID_ARG = 1,   /* NULL where a pointer is required, bad enum, n <= 0 ...          */
  DC_ERR_SHAPE = 2,         /* layer shapes do not connect, kernel larger than padded image    */
  DC_ERR_UNSUPPORTED = 3,   /* even k, groups other than 1 or c, shape outside a kernel's range */
  DC_ERR_NOT_MERGEABLE = 4, /* skip group without stride 1, c_in == c_out and 2p == k-1        */
  DC_ERR_WORKSPACE = 5,     /* workspace missing or too small                                  */
  DC_ERR_ALIGNMENT = 6,     /* a tensor pointer is not 16-byte aligned                         */
  DC_ERR_CUDA = 7,          /* a CUDA runtime/driver call failed                               */
  DC_ERR_TIMEOUT = 8        /* a bounded device-side wait ran out                              */
} dc_status;

typedef enum { DC_F32 = 0, DC_BF16 = 1 } dc_dtype;
typedef enum { DC_ACT_IDENTITY = 0, DC_ACT_RELU6 = 1 } dc_act;
typedef enum { DC_ALGO_AUTO = 0, DC_ALGO_TCGEN05 = 1, DC_ALGO_SIMT = 2 } dc_algo;

/* One convolution of a run, optionally followed by an eval-mode batch-norm (Sec. 3: f_theta_l). */
typedef struct {
  int c_in, c_out, groups;   /* groups == 1 dense; groups == c_in == c_out depthwise            */
  int k, stride, pad;
  const float *weight;       /* device, fp32 [c_out][c_in/groups][k][k]                         */
  const float *bias;         /* device, fp32 [c_out], or NULL                                   */
  const float *bn_gamma, *bn_beta, *bn_mean, *bn_var; /* device fp32 [c_out]; all NULL: no BN   */
  float bn_eps;
} dc_layer;

/* Skip addition y = run[first..last](x) + x inside a run (App. E.1).  Groups are disjoint and
 * listed in increasing order. */
typedef struct { int first, last; } dc_residual;

/* Geometry of one convolution (merged or not). */
typedef struct { int c_in, c_out, groups, k, stride, pad; } dc_geom;

/* An unmerged inverted-residual block: expand 1x1 (optional) -> depthwise -> project 1x1 (+x). */
typedef struct {
  int c_in, c_hidden, c_out;
  int has_expand;            /* 0: the block starts at the depthwise layer (c_hidden == c_in)   */
  int dw_k, dw_stride, dw_pad;
  int has_residual;          /* add the block input to the projection (stride 1, c_in == c_out) */
  dc_act act_expand, act_dw; /* activation after expand and after depthwise                     */
  const void *w_expand;      /* packed by dc_pack_weights for the call's dtype, or NULL         */
  const float *b_expand;
  const float *w_dw;         /* packed depthwise weights fp32 [k][k][c_hidden]                  */
  const float *b_dw;
  const void *w_project;     /* packed by dc_pack_weights for the call's dtype                  */
  const float *b_project;
} dc_block;

const char *dc_status_string(dc_status s);

/*
 * BN fusion (Sec. 2 "TensorRT", Sec. 5.1 "Evaluation"): w_out[o,.] = g[o]*W[o,.],
 * b_out[o] = beta[o] + (bias[o] - mean[o])*g[o], g = gamma/sqrt(var + eps); without BN it copies
 * W and the bias (zeros if NULL).  w_out: device fp32, same shape as layer->weight; b_out: device
 * fp32 [c_out].  fp32 arithmetic.
 */
dc_status dc_fold_bn(const dc_layer *layer, float *w_out, float *b_out, dc_stream stream);

/*
 * Host only: geometry of the merged convolution of a run (Sec. 3, Eq. 1) and the bytes of
 * device workspace dc_merge_chain needs for it.  k' = k1 + (k2-1) s1, s' = s1 s2,
 * p' = p1 + p2 s1, folded along the run.  Checks that shapes connect (DC_ERR_SHAPE), that
 * each skip group has stride 1, c_in == c_out and 2p == k-1 (DC_ERR_NOT_MERGEABLE, App. E.1),
 * odd k and groups in {1, c} (DC_ERR_UNSUPPORTED).  No device pointer is dereferenced.
 */
dc_status dc_merge_query(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                         dc_geom *merged, size_t *workspace_bytes);

/* Host only: bytes of the packed-weight buffer dc_conv_forward / dc_dwconv_forward read for a
 * convolution of this geometry and dtype. */
dc_status dc_packed_bytes(const dc_geom *g, dc_dtype dtype, size_t *bytes);

/*
 * Merge a run of convolutions whose intermediate activations are identities into one
 * convolution (Sec. 3; Eq. 1; App. E.1 for skips; App. E.2: the result equals the run with
 * all its zero padding applied before the first layer).  BN is folded per layer, depthwise
 * layers act as diagonal kernels, each skip group is merged first and gets an identity tap at
 * its centre, pieces are composed left to right:
 *   W'[o,i,u1+s1*u2,v1+s1*v2] += W2[o,c,u2,v2] * W1[c,i,u1,v1],  b' = b2 + (sum_taps W2) b1.
 * Outputs (device): w_merged fp32 [c_out][c_in][k'][k'], b_merged fp32 [c_out]; if w_packed is
 * not NULL also the packed copy for packed_dtype (size from dc_packed_bytes).  workspace: device,
 * at least the bytes dc_merge_query reports.  fp32 FMA arithmetic throughout.
 */
dc_status dc_merge_chain(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                         float *w_merged, float *b_merged, void *w_packed, dc_dtype packed_dtype,
                         void *workspace, size_t workspace_bytes, dc_stream stream);

/*
 * How dc_merge_chain walks a run.  DC_MERGE_STEPS: fold every layer, then compose the pieces
 * pairwise (one launch per step).  DC_MERGE_AUTO (what dc_merge_chain uses): as above, except
 * that every inverted-residual block inside the run -- dense 1x1 with stride 1, depthwise k x k,
 * dense 1x1 with stride 1, either a whole skip group or outside any -- is merged in one launch
 * straight from the raw layers (BN folded on the fly, the 6x wider intermediate kernel never
 * written): W'[o,i,t] = sum_c W3~[o,c] D~[c,t] W1~[c,i], which is Eq. 1 applied twice.  Both
 * forms evaluate the same formula in fp32; they differ in rounding order only.
 */
typedef enum { DC_MERGE_AUTO = 0, DC_MERGE_STEPS = 1 } dc_merge_algo;

/* As dc_merge_chain with the walk chosen by the caller (same workspace size for both). */
dc_status dc_merge_chain_algo(const dc_layer *layers, int n_layers, const dc_residual *res, int n_res,
                              float *w_merged, float *b_merged, void *w_packed, dc_dtype packed_dtype,
                              void *workspace, size_t workspace_bytes, dc_stream stream,
                              dc_merge_algo algo);

/*
 * dc_merge_chain for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for integration, it computes exactly what dc_merge_chain computes.)
 *
 * Who needs it: code that merges from inside an allocator or memory-pool callback, plug-ins whose
 * host forbids allocation calls once it is initialised, and processes that have handed all device
 * memory to another allocator -- none of them can cudaMalloc a workspace.  Here the intermediate
 * kernels of the merge live in a fixed array compiled into the library (dc_merge_chain_static_capacity()
 * bytes, 4 MiB; every GPU that loads the library holds it until the process exits).  The call
 * allocates and frees no device memory, itself or through any library (its host-side bookkeeping
 * uses a few small C++ vectors on the host heap).
 *
 * Inputs and outputs are as for dc_merge_chain, minus the workspace.  Runs whose intermediates
 * need more than the capacity (compare dc_merge_query's workspace_bytes) are refused with
 * DC_ERR_WORKSPACE before anything is launched.
 *
 * The first call on a device looks up the array's device address (with that device current); make
 * that first call before starting any stream capture.  All calls on a device share the one array:
 * it keeps the previous call's contents, which are overwritten (nothing needs to start at zero),
 * and two calls whose kernels overlap on the GPU (different streams, or a graph replayed
 * concurrently) race on it -- serialise them.
 */
dc_status dc_merge_chain_static(const dc_layer *layers, int n_layers, const dc_residual *res,
                                int n_res, float *w_merged, float *b_merged, void *w_packed,
                                dc_dtype packed_dtype, dc_stream stream);

/* Host only: size in bytes of the built-in scratch dc_merge_chain_static works in. */
size_t dc_merge_chain_static_capacity(void);

/*
 * Repack fp32 [c_out][c_in/groups][k][k] weights (device) into the layout the forward kernels
 * read.  Dense, DC_F32: fp32 [k][k][c_in][c_out].  Dense, DC_BF16: bfloat16 (round to nearest
 * even) in the K-chunked operand layout of the tensor-core kernel, zero padded (opaque; size
 * from dc_packed_bytes).  Depthwise, either dtype: fp32 [k][k][c].
 */
dc_status dc_pack_weights(const float *w, const dc_geom *g, dc_dtype dtype, void *w_packed,
                          dc_stream stream);

/* Host only: bytes of workspace dc_conv_forward needs (a status word plus padding). */
size_t dc_conv_workspace_bytes(void);

/*
 * Host only, launches nothing: name of the kernel dc_conv_forward would run for this problem
 * ("k_conv_tc_pairrows", "k_conv_tc_rows", "k_conv_tc_fold", "k_conv_tc", "k_conv_stem_tc", "k_conv_smallcin_bf16",
 * "k_conv_dense_bf16", "k_conv_dense_f32"), or NULL when the
 * geometry is invalid.  For reports (which kernel a timing belongs to); the string is static.
 */
const char *dc_conv_kernel_name(int n, int h, int w, const dc_geom *g, dc_dtype dtype);

/*
 * Forward pass of one dense convolution (the merged layer f_{theta^_i} of Eq. 1, or an
 * unmerged 1x1 / stem / head layer):  y = act(conv(x) + bias + residual).
 * x: [n][h][w][c_in], y: [n][h_out][w_out][c_out], residual: same shape as y or NULL, all of
 * `dtype`; w_packed from dc_merge_chain / dc_pack_weights for the same dtype; bias fp32 [c_out]
 * or NULL.  DC_BF16 runs as an implicit GEMM on the tensor cores (fp32 accumulate) when the
 * shape allows (c_in, c_out multiples of 8, stride 1 or 2, ...), else on CUDA cores; DC_F32
 * runs on CUDA cores in fp32.  workspace: device, >= dc_conv_workspace_bytes(), zeroed once by
 * the caller.
 */
dc_status dc_conv_forward(const void *x, int n, int h, int w, const dc_geom *g, const void *w_packed,
                          const float *bias, dc_act act, const void *residual, void *y,
                          dc_dtype dtype, void *workspace, size_t workspace_bytes, dc_stream stream);

/* As dc_conv_forward with the kernel family forced; DC_ERR_UNSUPPORTED if it cannot run the shape. */
dc_status dc_conv_forward_algo(const void *x, int n, int h, int w, const dc_geom *g,
                               const void *w_packed, const float *bias, dc_act act,
                               const void *residual, void *y, dc_dtype dtype, void *workspace,
                               size_t workspace_bytes, dc_stream stream, dc_algo algo);

/*
 * Forward pass of one depthwise convolution (the layers the merge leaves alone):
 * y[n,Y,X,c] = act( bias[c] + sum_{u,v} w[u][v][c] * x[n, Y*s+u-p, X*s+v-p, c] ).
 * w: fp32 [k][k][c] (dc_pack_weights with groups == c), bias fp32 [c] or NULL.
 */
dc_status dc_dwconv_forward(const void *x, int n, int h, int w, int c, int k, int stride, int pad,
                            const float *w_packed, const float *bias, dc_act act, void *y,
                            dc_dtype dtype, dc_stream stream);

/*
 * Synchronises `stream`, then returns DC_ERR_TIMEOUT if the bounded wait of a depthwise launch
 * (which takes no workspace to latch it in) ran out on the current device since the last call,
 * DC_OK otherwise; clears the flag.
 */
dc_status dc_dwconv_status(dc_stream stream);

/* Host only: workspace bytes dc_block_forward needs for this input size. */
dc_status dc_block_workspace_bytes(int n, int h, int w, const dc_block *blk, dc_dtype dtype,
                                   size_t *bytes);

/*
 * Forward pass of one unmerged inverted-residual block: expand 1x1 + act, depthwise + act,
 * project 1x1, plus the block input when has_residual (the skip addition that stays explicit
 * when the block is not merged into a single convolution, App. E.1).
 */
dc_status dc_block_forward(const void *x, int n, int h, int w, const dc_block *blk, void *y,
                           dc_dtype dtype, void *workspace, size_t workspace_bytes,
                           dc_stream stream);

/*
 * Synchronises `stream`, then returns the status latched in the first word of `workspace`
 * (DC_OK or DC_ERR_TIMEOUT) and clears it.
 */
dc_status dc_workspace_status(void *workspace, dc_stream stream);

/*
 * As dc_workspace_status; also returns, when not NULL, the code of the wait that gave up (`where`:
 * role in the upper bits, barrier index in the lower; 0 when nothing timed out) and the header's
 * first detail word.
 */
dc_status dc_workspace_status_where(void *workspace, dc_stream stream, unsigned int *where,
                                    unsigned int *detail);

/*
 * Self-test of the bounded waits (no counterpart in the paper): enqueues a one-CTA kernel whose two
 * roles wait, with the library's own wait routines, on a barrier that nothing completes.  After
 * limit_us microseconds (1..100000) the waits give up, DC_ERR_TIMEOUT and the site code 0x90000 are
 * latched in the workspace header, the second role leaves through the abort flag, and the kernel
 * returns normally; the detail word then holds the number of roles that left their wait (2).  No
 * copy or tensor-core work is in flight and nothing faults: the context stays usable, and the same
 * workspace serves ordinary launches again once dc_workspace_status has cleared it.
 * workspace: device, >= 256 bytes, 16-byte aligned.
 */
dc_status dc_selftest_bounded_wait(void *workspace, size_t workspace_bytes, unsigned int limit_us,
                                   dc_stream stream);

/*
 * Host only: the layout in which dc_chain_forward_host keeps a run's parameters on the device:
 * offsets[6 * i + j] is the byte offset of array j of layer i (j = 0 weight, 1 bias, 2 bn_gamma,
 * 3 bn_beta, 4 bn_mean, 5 bn_var; each rounded up to 256 bytes), total the size of the block.
 * A caller whose HOST arrays lie in one (pinned) block in exactly this layout, starting with layer
 * 0's weights, gets them copied with a single transfer instead of one per array; absent arrays
 * (NULL) keep their slot.  offsets may be NULL.  Only the layers' shapes are read.
 */
dc_status dc_chain_host_param_layout(const dc_layer *layers, int n_layers, size_t *offsets, size_t *total);

/* Host only: bytes of device workspace dc_chain_forward_host needs. */
dc_status dc_chain_host_workspace_bytes(const dc_layer *layers, int n_layers, const dc_residual *res,
                                        int n_res, int n, int h, int w, dc_dtype dtype,
                                        size_t *bytes);

/*
 * The whole path from HOST buffers: copy the run's parameters and the input to the device,
 * merge the run (dc_merge_chain), run the merged convolution (dc_conv_forward) and copy the
 * output back.  In `layers` every pointer is a HOST pointer here.  x_host / y_host: host
 * NHWC buffers of `dtype` (pinned memory makes the copies asynchronous).  workspace: device.
 * Synchronises the stream before returning.
 */
dc_status dc_chain_forward_host(const dc_layer *layers, int n_layers, const dc_residual *res,
                                int n_res, const void *x_host, int n, int h, int w, dc_act act,
                                void *y_host, dc_dtype dtype, void *workspace,
                                size_t workspace_bytes, dc_stream stream);

/*
 * The same without the final synchronisation: everything (copies in, merge, forward, copy out) is
 * queued on `stream` and the call returns.  The host buffers, the layers' host arrays and the
 * workspace must stay untouched until the stream has passed this point (y_host is valid after the
 * caller has synchronised the stream or an event recorded behind the call).  With pinned host
 * buffers and one workspace per stream, calls on different streams overlap their copies in both
 * directions with each other's kernels: Sec. 5's deployment setting of a stream of input batches.
 */
dc_status dc_chain_forward_host_async(const dc_layer *layers, int n_layers, const dc_residual *res,
                                int n_res, const void *x_host, int n, int h, int w, dc_act act,
                                void *y_host, dc_dtype dtype, void *workspace,
                                size_t workspace_bytes, dc_stream stream);

/* ---------------------------------------------------------------------------------------------
 * The selector's two dynamic programmes (Sec. 4.3).  Host only: every pointer is host memory, no
 * device call is made.  Boundaries are 0..L for a network of L layers; tables are row-major
 * (L+1) x (L+1) and only entries [i][j] with i < j are read.
 * ------------------------------------------------------------------------------------------- */

/* Latency of a span that cannot be merged into one convolution; sums that contain it stay at it. */
#define DC_DP_INF (1ll << 60)

/*
 * Algorithm 1 (Eq. 6a, 6b): T_opt[k][l] = min over S in {k+1..l-1} of the summed latency
 * T[s_{i-1}][s_i] of the pieces (k, s_1], ..., (s_n, l], with T_opt[k][k] = 0.
 * T: integer latencies (any unit), DC_DP_INF where layers i+1..j do not merge.
 * T_opt: out, (L+1) x (L+1).  split: out, (L+1) x (L+1) ints; split[k][l] = m is the last boundary
 * of the optimal pattern of (k, l] (m == k: one merged layer), so that
 * S_opt[k][l] = S_opt[k][m] + {m}; ties take the smallest m.  Entries with k >= l are set to 0 / k.
 * DC_ERR_INVALID_ARG for NULL pointers, L <= 0 or a negative latency.
 */
dc_status dc_dp_optimal_latency(const long long *T, int L, long long *T_opt, int *split);

/* Host only: writes S_opt[k][l] (increasing) into S (room for L ints) and its size into n_S, from
 * the split table of dc_dp_optimal_latency. */
dc_status dc_dp_pattern(const int *split, int L, int k, int l, int *S, int *n_S);

/*
 * Algorithm 2 (Eq. 5, 7, 8): the activations to keep (A) and the boundaries that stay after merging
 * (S, A a subset of S) that maximise the summed importance I[a_{j-1}][a_j] of the blocks of A under
 * "summed latency of the pieces of S < T0" (strict).  I: doubles, -infinity excludes a block.
 * A, S: out, increasing, room for L ints each; objective: out, D[L][T0]; feasible: out, 0 when no
 * pattern meets the budget (T0 <= T_opt[0][L]) or every pattern contains an excluded block -- A and
 * S are then empty.  Ties take the smallest k.  Memory: (L+1)(T0+1) doubles and ints on the host
 * heap; DC_ERR_WORKSPACE if that cannot be allocated, DC_ERR_INVALID_ARG for bad arguments.
 */
dc_status dc_dp_select(const long long *T, const double *I, int L, long long T0, int *A, int *n_A,
                       int *S, int *n_S, double *objective, int *feasible);

/*
 * Extended selector (App. B).  A block (i, j] now carries the indicators d_i, d_j of a non-linear
 * activation at its two ends, and its importance is I[i][j][d_i][d_j], stored as doubles at
 * ((i * (L+1) + j) * 2 + d_i) * 2 + d_j.  sigma_id[p], p = 0..L (0 or 1), says whether the original
 * activation at boundary p is an identity (p = 0: the network input).  Before either programme runs,
 * the blocks that App. B excludes count as -infinity: d = 0 at an end whose original activation is
 * non-linear, and d_j = 0 when both ends are identities in the original network (App. B.2).
 *
 * Algorithm 3: I_opt[k][l][a][b] = best summed importance of a chain of blocks from boundary k to
 * boundary l with d_k = a, d_l = b and d = 0 at every inner boundary of the chain.  split (ints, same
 * indexing) holds the chain's last inner boundary m (m == k: the single block), so that
 * B_opt[k][l][a][b] = B_opt[k][m][a][0] + {m}; ties take the smallest m.  The listing's update is
 * read with the maximiser m where it prints m', and its m' = k term as the single block
 * I[k][l][a][b].  DC_ERR_INVALID_ARG for NULL pointers, L <= 0 or a flag other than 0 / 1.
 */
dc_status dc_dp_optimal_importance(const double *I, const unsigned char *sigma_id, int L, double *I_opt, int *split);

/* Host only: writes B_opt[k][l][a][b] (increasing) into B (room for L ints) and its size into n_B,
 * from the split table of dc_dp_optimal_importance. */
dc_status dc_dp_importance_pattern(const int *split, int L, int k, int l, int a, int b, int *B, int *n_B);

/* App. B.3, in place: every block's importance (j > i) loses alpha times the mean of the n_deltas
 * accuracy changes measured on the size-one blocks.  DC_ERR_INVALID_ARG for NULL or n_deltas <= 0. */
dc_status dc_dp_normalize_importance(double *I, int L, const double *deltas, int n_deltas, double alpha);

/*
 * Algorithm 4 (the extended surrogate problem of App. B): boundaries B of the importance blocks,
 * the kept non-linear activations A (a subset of B and of S), the boundaries S that stay after
 * merging, and the indicators of the network's two ends, maximising the summed
 * I[b'][b][1_A(b')][1_A(b)] over the blocks of B under "summed latency of the pieces of S < T0".
 * The state is D[l][t][a] with a = d_l; S and B carry that index like A, and the result is read at
 * a_last = argmax_a D[L][T0][a] (where the listing prints A).  A, S, B: out, increasing, room for L
 * ints each; d_first, d_last: out, d_0 and d_L; objective, feasible as for dc_dp_select.  Ties take
 * the smallest k, then alpha = 0, then a = 0.  Memory: 2 (L+1)(T0+1) doubles and ints on the host
 * heap (DC_ERR_WORKSPACE if that fails).
 */
dc_status dc_dp_select_ext(const long long *T, const double *I, const unsigned char *sigma_id, int L, long long T0,
                           int *A, int *n_A, int *S, int *n_S, int *B, int *n_B, int *d_first, int *d_last,
                           double *objective, int *feasible);

#ifdef __cplusplus
}
#endif
#endif /* DC_H_ */

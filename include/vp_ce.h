/*
 * vp_ce.h -- C ABI of the fused vocabulary projection + cross-entropy library (sm_100a).
 *
 * The operation (paper section 3.2, Eq. 2; Appendix C, Algorithm 3): logits Y = H * W^T are
 * formed one vocabulary shard ("strip") at a time; every strip is folded into a per-token
 * running state S = (m, z, y_t) and dropped, so the tokens x vocabulary matrix never exists.
 * After all shards the negative log-likelihood of a token is m + log z - y_t.  Backward
 * replays the same meetings from the saved normaliser lse = m + log z, forms the softmax
 * residual of one strip at a time and contracts it into the input and weight gradients.
 * On one device the ring of Algorithm 3 is a loop over shards: token chunk c (global index
 * chunk_index_base + local chunk) meets shard q_i = (c - i) mod P at step i = 0..P-1, with
 * P = ceil(V / block_v).
 *
 * Conventions for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller unless a parameter is
 *     explicitly called "host".  Inputs are never written.  The library allocates and
 *     frees no device memory in these calls; scratch memory is the caller's `workspace`.
 *   - Layouts (row-major, no padding):
 *       H      [T, d]  bfloat16      hidden states
 *       W      [V, d]  bfloat16      projection weight (logits = H * W^T)
 *       labels [T]     int32         target ids in [0, V) or ignore_index
 *       loss, lse, dloss [T] float32
 *       dH     [T, d]  bfloat16      dW [V, d] float32
 *   - H, W, dH, dW and workspace must be 16-byte aligned; d must be a multiple of 8;
 *     block_v must be a multiple of 256 and T_chunk a multiple of 128 (tile shapes).
 *   - `stream` is a cudaStream_t passed as void*.  Calls are asynchronous on that stream
 *     and do not synchronise with the host.  The return value reports host-detectable
 *     errors only; conditions found on the device (a label outside [0, V) that is not
 *     ignore_index; a bounded wait inside a kernel that ran out) set a status word in the
 *     workspace, read back with vp_ce_device_status.
 *   - T == 0 (an empty batch) is accepted by vp_ce_forward and vp_ce_backward: nothing is launched;
 *     the backward zeroes dW when accumulate_dW == 0.  Other non-positive sizes are VPCE_INVALID_ARG.
 *   - A token whose label equals ignore_index has loss 0 and a zero gradient row; its lse
 *     is still computed.  A label outside [0, V) is treated the same way and flagged.
 */
#ifndef VP_CE_H_
#define VP_CE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int vpce_status;
#define VPCE_OK                  0
#define VPCE_INVALID_ARG         1  /* null pointer, non-positive size                        */
#define VPCE_UNSUPPORTED         2  /* alignment or divisibility rule above not met           */
#define VPCE_WORKSPACE_TOO_SMALL 3
#define VPCE_CUDA_ERROR          4  /* a CUDA runtime/driver call or a launch failed          */
#define VPCE_STATIC_SCRATCH_EXCEEDED 5  /* vp_ce_forward_static: sizes beyond its built-in scratch */

/* Bits of the device status word (vp_ce_device_status). */
#define VPCE_DEV_LABEL_OUT_OF_RANGE 1
#define VPCE_DEV_WAIT_EXPIRED       2

/*
 * Bytes of workspace needed by vp_ce_forward / vp_ce_backward for a given token chunk,
 * hidden width and shard width.  Depends on neither V nor T (Eq. 1 of section 3.2: the live
 * logit memory is O(N V / P) = O(T_chunk * block_v)).  Pure host arithmetic; returns 0 for
 * arguments that the other calls would reject.
 */
size_t vp_ce_workspace_bytes(int64_t T_chunk, int64_t d, int64_t block_v);

/*
 * Forward (Algorithm 3 with Fold = Eq. 2, output line "m + log z - y").
 * Writes lse[n] for every token and loss[n] = lse[n] - y[n, labels[n]] (0 if ignored).
 * T_chunk: tokens per internal chunk (the paper's per-rank batch N); chunk c covers tokens
 * [c*T_chunk, min(T, (c+1)*T_chunk)).  chunk_index_base: global index of this call's first
 * chunk (rotation of the shard order when a long stream is cut into several calls).
 * The workspace contents are undefined on entry and on return except for the status word,
 * which this call clears first.
 */
vpce_status vp_ce_forward(const void* H, const void* W, const int32_t* labels,
                          int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                          float* loss, float* lse,
                          int64_t T_chunk, int64_t chunk_index_base,
                          void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward (Appendix C: replay the meetings from the saved per-token normaliser).
 * lse: the forward's output.  dloss: per-token upstream gradient of loss[n], or NULL for
 * the masked mean (1 / n_valid on valid tokens, n_valid counted from labels; 0 valid tokens
 * give zero gradients).  dH is overwritten.  dW is overwritten when accumulate_dW == 0 and
 * added to otherwise (fp32 accumulation across calls of a streamed context).
 * Either dH or dW (not both) may be NULL: that gradient and its contraction are skipped
 * (a frozen projection weight, or an input that needs no gradient).
 * The residual strip is staged as bf16, but the target entry of every token's row is applied
 * exactly: what rounding took from it is added back to dH and dW in fp32, in a fixed order, so
 * results are bitwise reproducible and the one-hot part of the gradients carries no rounding bias.
 */
vpce_status vp_ce_backward(const void* H, const void* W, const int32_t* labels, const float* lse,
                           const float* dloss, void* dH, float* dW,
                           int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                           int64_t T_chunk, int64_t chunk_index_base, int accumulate_dW,
                           void* workspace, size_t workspace_bytes, void* stream);

/*
 * Single meetings, for a ring driver that runs Algorithm 3 ACROSS devices (each rank holds its own batch
 * X_r [N, d] with targets t_r and owns shard W_r, the rows [v_lo, v_lo + shard_rows) of the weight; either
 * the shard or the batch travels around the ring, section 3.2 "Which tensor travels").  One call = one
 * meeting of a batch with a shard; everything it touches is in this device's memory.
 *
 * vp_ce_meeting_forward: forms the strip X W_shard^T and folds it into the batch's running state (Eq. 2;
 * Algorithm 3, Fold).  state is the caller's DEVICE array [3][N] fp32 = (m, z, y_t): it stays on the rank in
 * the move-weights schedule and travels with (X, t) in the move-activations schedule.  first != 0: the
 * state starts from (-inf, 0, 0) (its previous contents are ignored) and the status word is cleared;
 * last != 0: lse[n] = m + log z and loss[n] = lse[n] - y_t (0 if ignored) are written as well.
 * shard_rows and N need not be multiples of the tile shapes.
 *
 * vp_ce_meeting_backward: the backward meeting (Appendix C), in up to three phases selected by `phases`
 * so that a ring driver can wait for a travelling accumulator between them:
 *   VPCE_PHASE_RESIDUAL     recompute the strip, residual G = dloss (exp(Y - lse) - onehot) -> workspace
 *   VPCE_PHASE_INPUT_GRAD   dX_acc (+)= G W_shard   fp32 [N, d]; first != 0 overwrites; last != 0 writes the
 *                           final bf16 dX [N, d] instead of the accumulator (dX_acc is read unless first)
 *   VPCE_PHASE_WEIGHT_GRAD  dW_shard (+)= G^T X     fp32 [shard_rows, d]; accumulate_dW == 0 overwrites
 * The gradient of the tensor that travels goes with it: dX_acc in the move-activations schedule, dW_shard
 * in the move-weights schedule.  Phases of one meeting must use the same workspace, in this order, with
 * nothing else using it in between.  dloss is required (the ring driver knows the global token count).
 *
 * vp_ce_meeting_workspace_bytes(N, d, shard_rows): bytes both calls need (O(N * shard_rows), Eq. 1).
 */
#define VPCE_PHASE_RESIDUAL    1
#define VPCE_PHASE_INPUT_GRAD  2
#define VPCE_PHASE_WEIGHT_GRAD 4
size_t vp_ce_meeting_workspace_bytes(int64_t N, int64_t d, int64_t shard_rows);
vpce_status vp_ce_meeting_forward(const void* X, const void* W_shard, const int32_t* targets,
                                  int64_t N, int64_t d, int64_t shard_rows, int64_t v_lo, int64_t V,
                                  int32_t ignore_index, float* state, int first, int last,
                                  float* loss, float* lse, void* workspace, size_t workspace_bytes, void* stream);
vpce_status vp_ce_meeting_backward(const void* X, const void* W_shard, const int32_t* targets, const float* lse,
                                   const float* dloss, int64_t N, int64_t d, int64_t shard_rows, int64_t v_lo,
                                   int64_t V, int32_t ignore_index, int phases, float* dX_acc, int first, int last,
                                   void* dX, float* dW_shard, int accumulate_dW,
                                   void* workspace, size_t workspace_bytes, void* stream);

/*
 * Masked mean of the per-token loss (not part of the paper's operator, which outputs
 * per-token values; this is the reduction the benchmark's metric is stated on).
 * mean_out[0] = sum of loss over valid tokens / n_valid (0 when n_valid == 0);
 * n_valid_out[0] = n_valid.  Both are device pointers.  Deterministic (fixed order).
 * T == 0 is accepted (mean 0, n_valid 0; loss and labels may then be NULL).
 */
vpce_status vp_ce_mean_loss(const float* loss, const int32_t* labels, int64_t T, int64_t V,
                            int32_t ignore_index, float* mean_out, int32_t* n_valid_out, void* stream);

/*
 * Gradient of that masked mean with respect to the per-token loss (chain rule for callers that
 * differentiate through vp_ce_mean_loss; not in the paper): dloss_out[n] = upstream / n_valid for
 * valid tokens and 0 for the others.  n_valid is the DEVICE int32 that vp_ce_mean_loss wrote,
 * upstream a DEVICE float (NULL means 1).  n_valid == 0 gives all zeros.  T == 0 launches nothing.
 */
vpce_status vp_ce_mean_loss_grad(const int32_t* labels, int64_t T, int64_t V, int32_t ignore_index,
                                 const int32_t* n_valid, const float* upstream, float* dloss_out, void* stream);

/*
 * Copies the device status word of `workspace` to host_out[0] (HOST pointer) and
 * synchronises `stream`.  0 means no device-side condition was seen since the last
 * vp_ce_forward / vp_ce_backward call on this workspace began: each of those two calls clears the
 * word first, so a caller that runs them back to back and wants the forward's conditions reads the
 * word in between.  vp_ce_fwd_bwd_host clears it once, before its forward half, and the word read
 * after it covers the whole pass.  Both passes flag a label outside [0, V).
 */
vpce_status vp_ce_device_status(const void* workspace, int32_t* host_out, void* stream);

/* Static, NUL-terminated description of a status code. */
const char* vp_ce_status_string(vpce_status s);

/* Number of kernels the library launched on behalf of the caller since the process
 * started (monotonic, host-side counter; used by the benchmark's launch accounting). */
int64_t vp_ce_launch_count(void);

/*
 * One whole pass (Algorithm 3 forward, then the Appendix C backward with the masked-mean
 * upstream gradient) for callers whose activations live in HOST memory.
 *   H_host [T, d] bf16, labels_host [T] int32          HOST, read (pinned memory makes the
 *   loss_host [T] fp32, dH_host [T, d] bf16            HOST, written    copies asynchronous)
 *   W [V, d] bf16, dW [V, d] fp32                      DEVICE: the weight and its gradient
 *                                                      accumulator stay resident, as in training
 *   H_dev, labels_dev, loss_dev, lse_dev, dH_dev       DEVICE staging buffers of the same shapes,
 *                                                      owned by the caller; nothing is allocated here
 * Copies H and labels to the device, runs vp_ce_forward and vp_ce_backward (dloss = NULL), copies
 * loss and dH back, then synchronises `stream`, so the host buffers are valid on return.
 * Errors are those of the two calls it wraps.
 */
vpce_status vp_ce_fwd_bwd_host(const void* H_host, const int32_t* labels_host, const void* W, float* loss_host,
                               void* dH_host, float* dW, int64_t T, int64_t d, int64_t V, int64_t block_v,
                               int32_t ignore_index, int64_t T_chunk, int64_t chunk_index_base, int accumulate_dW,
                               void* H_dev, int32_t* labels_dev, float* loss_dev, float* lse_dev, void* dH_dev,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Forward for callers that can neither allocate device memory nor hand over a workspace.
 * (The paper has no counterpart: its operator runs under a framework allocator.)
 *
 * Some callers of this library run where cudaMalloc is off limits: a plug-in that executes
 * inside another runtime's memory plan (every device byte is owned by that runtime's arena and
 * the plug-in may only touch the tensors it is handed), a step of a latency-critical serving
 * loop where an allocation would synchronise the device, or code that runs after the process
 * has deliberately filled the GPU.  For them this entry point computes exactly what
 * vp_ce_forward computes, with the same kernels, but its scratch memory (per-token running
 * state, per-tile partial states, status word) is a fixed array compiled into the library:
 * VPCE_STATIC_SCRATCH_BYTES bytes of device memory that every GPU which loads the library
 * holds until the process exits.
 *
 *   - Inputs and outputs are the caller's, as for vp_ce_forward.  device_status_out is an
 *     optional DEVICE int32 that receives the status word (the bits VPCE_DEV_*) at the end of
 *     the call; pass NULL to skip it.
 *   - Limit: the forward part of the workspace layout for (T_chunk, block_v) must fit the
 *     array, roughly 8 * T_chunk * (block_v / 256 + 2) bytes; T_chunk = 4096 with
 *     block_v = 8192 fits.  Larger sizes return VPCE_STATIC_SCRATCH_EXCEEDED and launch
 *     nothing; T, V and d are not limited by it.
 *   - No cudaMalloc, cudaFree, event or stream creation or other allocating routine is called.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents; the call
 *     clears what must start at zero itself.  Two calls that overlap on the GPU (different
 *     streams, or different host threads without ordering) race on it and give wrong results:
 *     order them on one stream or with events.
 */
#define VPCE_STATIC_SCRATCH_BYTES (1280u * 1024u)
vpce_status vp_ce_forward_static(const void* H, const void* W, const int32_t* labels,
                                 int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                                 float* loss, float* lse, int64_t T_chunk, int64_t chunk_index_base,
                                 int32_t* device_status_out, void* stream);

/*
 * FP32-input variants (TF32 tensor cores, fp32 accumulation): the precision of the paper's isolated
 * Ring-DTP benchmark (Appendix C states FP32; whether its matmuls used TF32 is not stated).  Same
 * method, semantics, status codes and workspace rules as vp_ce_forward / vp_ce_backward, except:
 *   H [T, d], W [V, d] are float32; dH [T, d] is float32 (it also serves as the running
 *   accumulator across shards); the residual strip in the workspace is float32, so
 *   vp_ce_workspace_bytes_f32 is about twice as large minus the separate accumulator;
 *   d must be a multiple of 32.  The tensor core reads the upper 19 bits of each input.
 */
size_t vp_ce_workspace_bytes_f32(int64_t T_chunk, int64_t d, int64_t block_v);
vpce_status vp_ce_forward_f32(const float* H, const float* W, const int32_t* labels,
                              int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                              float* loss, float* lse, int64_t T_chunk, int64_t chunk_index_base,
                              void* workspace, size_t workspace_bytes, void* stream);
vpce_status vp_ce_backward_f32(const float* H, const float* W, const int32_t* labels, const float* lse,
                               const float* dloss, float* dH, float* dW,
                               int64_t T, int64_t d, int64_t V, int64_t block_v, int32_t ignore_index,
                               int64_t T_chunk, int64_t chunk_index_base, int accumulate_dW,
                               void* workspace, size_t workspace_bytes, void* stream);

/*
 * Watchdog of the kernels (no counterpart in the paper).  Every wait inside a kernel (on a copy, on
 * the tensor cores, on another warp or on the other CTA of a pair) is bounded: when it has lasted
 * longer than the limit the CTA stops taking work, waits (bounded again) for what it still has in
 * flight, releases its tensor memory and returns, and VPCE_DEV_WAIT_EXPIRED is set in the status
 * word; the outputs of that call are then undefined, the context stays usable and the next call
 * starts clean.  vp_ce_set_wait_limit_ns sets the limit for all later launches of this process
 * (clamped to [1 ms, 60 s]; ns <= 0 changes nothing) and returns the previous value.  The default
 * is 2 s.  A kernel that gives up can take up to about twice the limit to return.
 */
int64_t vp_ce_set_wait_limit_ns(int64_t ns);

/*
 * Tuning knob (no counterpart in the paper).  When the 256 x 256 output tiles of a gradient GEMM
 * do not fill a whole number of rounds of the CTA pairs, the remainder tiles are run as two or
 * three parts along the contracted dimension; the parts of a tile add into the output in the order
 * of their index (flags in the workspace), so results stay bitwise reproducible for a given
 * setting.  vp_ce_set_tail_parts(parts) overrides the library's choice for all later launches of
 * this process: -1 = the library decides per launch geometry (default), 0 = never split,
 * 2..8 = the remainder tiles in that many parts whenever the contraction is long enough.  Other
 * values change nothing.  Returns the previous setting.  Results of different settings differ in
 * the last bits (another summation order).
 */
int vp_ce_set_tail_parts(int parts);

/*
 * The decision the library takes for a gradient GEMM of the given launch geometry (pure host
 * arithmetic, no device needed): row_tiles x col_tiles output tiles of 256 x 256 handed out to
 * `pairs` CTA pairs in raster groups of group_cols column tiles, the last column tile with an MMA
 * width of last_width (<= 256), k_blocks k-blocks (of 64 bf16 / 32 fp32 elements) in the
 * contraction.  Outputs: how many tiles at the end of the work list are split, into how many
 * parts, and by how many k-blocks each part is longer than the one before it (0 tiles = no
 * split).  Honours vp_ce_set_tail_parts.  Returns VPCE_INVALID_ARG for non-positive arguments.
 */
vpce_status vp_ce_tail_choice(int row_tiles, int col_tiles, int group_cols, int last_width, int k_blocks, int pairs,
                              int* n_tiles_split, int* parts, int* stagger);

/*
 * TEST HOOK (no counterpart in the paper): makes one copy of the next launch "get lost" so that
 * the give-up path above can be exercised without any invalid access.  The next launch of kernel
 * kind `kernel_kind` (0 forward strip, 1 backward strip, 2 input-gradient GEMM, 3 weight-gradient
 * GEMM) does not issue the operand copies of k-block `k_block` of the first tile of its work list
 * in the CTAs named by `cta_ranks` (bit 0: the single CTA or the leader of a CTA pair, bit 1: the
 * second CTA of a pair); the data simply never arrives.  One-shot: the launch that consumes it
 * disarms it.  kernel_kind < 0 disarms.  Returns VPCE_INVALID_ARG for values out of range.
 */
vpce_status vp_ce_debug_drop_copy(int kernel_kind, int k_block, int cta_ranks);

/*
 * Measurement aid (no counterpart in the paper).  While enabled, every tensor-core kernel
 * launch is bracketed by two CUDA events on the launching stream.  vp_ce_profile_collect
 * waits for the recorded events, adds up the elapsed milliseconds and launch counts per kernel
 * kind into the HOST arrays ms_out[4], launches_out[4] (0 = forward strip + fold,
 * 1 = backward strip + residual, 2 = input-gradient GEMM, 3 = weight-gradient GEMM) and
 * forgets them.  Not thread-safe against concurrent launches from other host threads.
 */
void vp_ce_profile_enable(int on);
vpce_status vp_ce_profile_collect(double* ms_out, int64_t* launches_out);

#ifdef __cplusplus
}
#endif
#endif /* VP_CE_H_ */

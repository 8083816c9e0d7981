/*
 * stream_adamw.h -- C ABI of the bucket-streamed AdamW update (OffloadStreamAdamW; paper section 3.4 and the
 * appendix "OffloadStreamAdamW", Algorithm 4), part of the same library as vp_ce.h (sm_100a).
 *
 * The method: a rank's optimizer state (fp32 master weights, first and second moments) and its final gradients
 * live in HOST memory.  The flat parameter shard is cut into buckets of at most `bucket_params` parameters
 * (Algorithm 4, first line) that rotate through `slots` staging slots in device memory and three streams:
 * (i) host-to-device copy of a bucket's master weight, moments and gradient, (ii) one fused kernel that applies
 * the AdamW update in fp32 and refreshes the bf16 working weight, (iii) copy of the updated fp32 state back to
 * the host.  A slot is taken again only after its write-back has finished.  The three stages of different
 * buckets overlap, so a step costs about (number of buckets) x max(copy in, update, copy out)   (Eq. 4), and the
 * staging memory is slots x bucket_params x 16 bytes.  Inside a bucket the stages run piece by piece (up to 8 pieces
 * of at least 4 Mi parameters), so the update and write-back of a large bucket begin when its first piece has
 * arrived; the results do not depend on the bucketing (the rule is elementwise).
 *
 * The update of one parameter with gradient g at step t = 1, 2, ... (decoupled weight decay; the appendix says
 * the fused kernel keeps the reference implementation's bias correction, weight decay and update order):
 *     p <- p (1 - lr weight_decay);  m <- beta1 m + (1 - beta1) g;  v <- beta2 v + (1 - beta2) g^2;
 *     p <- p - lr (m / (1 - beta1^t)) / (sqrt(v / (1 - beta2^t)) + eps);      w = bf16(p)  (nearest even)
 * All arithmetic is fp32; 1 - beta^t and lr / (1 - beta1^t) are formed in double on the host.
 *
 * Status codes are those of vp_ce.h (0 ok, 1 invalid argument, 2 unsupported, 3 staging too small, 4 CUDA error).
 */
#ifndef STREAM_ADAMW_H_
#define STREAM_ADAMW_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct osadamw_ctx osadamw_ctx;

/* Device bytes of staging for `slots` slots of `bucket_params` parameters: each slot holds p, m, v, g in fp32
 * (M_stage = O(s beta), Eq. 4).  0 for non-positive arguments. */
size_t osadamw_staging_bytes(int64_t bucket_params, int slots);

/*
 * Creates a pipeline on the current device: three non-blocking streams (copy in, update, copy out) and the events
 * that order them.  `staging` is a DEVICE buffer of at least osadamw_staging_bytes(...) bytes, 256-byte aligned,
 * owned by the caller and lent to the pipeline until osadamw_destroy; no device memory is allocated here.
 * *out receives the handle.  Not thread-safe per handle; different handles are independent.
 */
int osadamw_create(osadamw_ctx** out, int64_t bucket_params, int slots, void* staging, size_t staging_bytes);

/* Waits for the pipeline's streams, destroys them and frees the handle.  NULL is accepted. */
int osadamw_destroy(osadamw_ctx* ctx);

/*
 * One optimizer step (Algorithm 4) over a flat shard of n parameters.
 *   master, m, v   HOST fp32 [n], read and overwritten with the updated state
 *   grad           HOST fp32 [n], read                     (pinned host memory makes the copies asynchronous
 *                                                           and lets copy-in, update and copy-out overlap)
 *   w_bf16         DEVICE bfloat16 [n], overwritten with the refreshed working weight
 *   bucket_offsets HOST int64 [n_buckets + 1] rising from 0 to n, every bucket at most bucket_params long
 *                  (a caller that groups whole tensors into buckets passes its boundaries), or NULL for
 *                  contiguous buckets of bucket_params parameters (n_buckets is then ignored)
 *   step           t >= 1
 *   user_stream    cudaStream_t as void*: work already enqueued there (e.g. the producer of the gradients'
 *                  host copy, earlier readers of w_bf16) is waited for before the first copy, and on return
 *                  the stream is made to wait for the last update kernel, so later work on it sees w_bf16.
 * The call only enqueues work and returns; the HOST arrays are complete after osadamw_wait.
 * The host arrays must not be touched between the call and osadamw_wait.  n == 0 is a no-op.
 */
int osadamw_step(osadamw_ctx* ctx, float* master, float* m, float* v, const float* grad, void* w_bf16,
                 int64_t n, const int64_t* bucket_offsets, int64_t n_buckets,
                 float lr, float beta1, float beta2, float eps, float weight_decay, int64_t step,
                 void* user_stream);

/* Blocks the host until every write-back of the steps enqueued so far has landed in host memory. */
int osadamw_wait(osadamw_ctx* ctx);

/*
 * The fused update alone on DEVICE-resident fp32 state (the kernel of stage (ii); p, m, v are updated in place,
 * w_bf16 [n] is written).  Asynchronous on `stream`.  p, m, v, g must be 16-byte aligned, w_bf16 8-byte aligned.
 */
int osadamw_update_device(float* p, float* m, float* v, const float* g, void* w_bf16, int64_t n,
                          float lr, float beta1, float beta2, float eps, float weight_decay, int64_t step,
                          void* stream);

#ifdef __cplusplus
}
#endif
#endif /* STREAM_ADAMW_H_ */

/*
 * loract.h -- C ABI of the LoRAct online activation-compression hot path for NVIDIA B200 (sm_100a).
 *
 * The library compresses a saved activation matrix X (n_tokens x d, row-major, bf16 or fp32) to a
 * rank-r factor pair (U, V) with the paper's sampling-based orthogonal decomposition (Algorithm 1),
 * and serves the backward-pass consumers from the factors.  Notation: the paper's A (m x n), k and t
 * are X (n_tokens x d), rank and power_iters here.
 *
 * Conventions common to every call
 *   - Every pointer named X, U, V, G, dW, gamma, beta, A_out, rstd, mean, idx_*, ws is a DEVICE pointer
 *     to memory the caller owns (allocate it with any CUDA allocator); the descriptor and the out_host
 *     arguments are HOST pointers.  The library allocates no device memory and frees none.
 *   - Matrices are row-major.  X has row stride ldx elements; U is n_tokens x rank (stride rank),
 *     V is rank x d (stride d).  U, V, X_out, A_out have X's dtype.  dW is always fp32.
 *   - Alignment: every matrix base pointer 16-byte aligned; d, ldx, ldg multiples of 8 (bf16) or
 *     4 (fp32) elements, so that every row starts on a 16-byte boundary.
 *   - rank: a multiple of 16, 16 <= rank <= 512, rank <= n_tokens and rank <= d.
 *   - Calls are asynchronous on the CUDA stream passed as `stream` (a cudaStream_t cast to void*;
 *     NULL is the default stream) and never synchronise, except loract_read_device_status.
 *   - Host-detectable errors return a status and launch nothing.  Conditions found on the device are recorded
 *     in a 32-bit word at the start of `ws`; read it with loract_read_device_status.  After a clamped pivot
 *     or a non-finite input the outputs are still fully written (finite where the input was).  After an
 *     expired wait (LORACT_DEV_WAIT_EXPIRED) the kernel that gave up has skipped its stores: the outputs
 *     are unspecified and must not be used.
 *   - `ws` is scratch of at least loract_workspace_bytes(desc) bytes, 256-byte aligned, private to one
 *     in-flight call.  The same (seed, call_id, n_tokens, rank) always selects the same rows.
 */
#ifndef LORACT_H_
#define LORACT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  LORACT_OK = 0,
  LORACT_ERR_INVALID_ARG = 1,
  LORACT_ERR_UNSUPPORTED = 2,
  LORACT_ERR_ALIGNMENT = 3,
  LORACT_ERR_WORKSPACE_TOO_SMALL = 4,
  LORACT_ERR_CUDA = 5,
  LORACT_ERR_NUMERIC = 6,
  LORACT_ERR_TIMEOUT = 7
} loract_status_t;

typedef enum { LORACT_F32 = 0, LORACT_BF16 = 1 } loract_dtype_t;
typedef enum { LORACT_NORM_RMS = 0, LORACT_NORM_LAYER = 1 } loract_norm_t;
typedef enum { LORACT_ACT_SILU = 0, LORACT_ACT_GELU = 1 } loract_act_t;

/* Bits of the device status word (see loract_read_device_status). */
#define LORACT_DEV_PIVOT_CLAMPED 0x1u  /* a Cholesky pivot was not positive and was clamped       */
#define LORACT_DEV_WAIT_EXPIRED  0x2u  /* a bounded device-side wait gave up; results are invalid */
#define LORACT_DEV_SAMPLER_SHORT 0x4u  /* the sampler could not find `rank` distinct rows          */
#define LORACT_DEV_NONFINITE     0x8u  /* a non-finite value reached the small-block factorisation */

typedef struct {
  int64_t n_tokens;      /* rows of X (the paper's m)                                        */
  int64_t d;             /* columns of X (the paper's n)                                     */
  int64_t ldx;           /* row stride of X in elements, >= d                                */
  int32_t rank;          /* r (the paper's k)                                                */
  int32_t power_iters;   /* t of Algorithm 1 (its loop), 0 <= t <= 8;     the paper's runs use 0   */
  int32_t dtype;         /* loract_dtype_t of X, U, V, X_out, A_out, G, gamma, beta          */
  int32_t reserved;      /* must be 0                                                        */
  uint64_t seed;         /* Philox key                                                       */
  uint64_t call_id;      /* Philox counter high words: distinguishes layer / step / rank     */
} loract_desc_t;

/* Bytes of scratch that loract_compress / loract_compress_prenorm / loract_weight_grad need for this
 * descriptor (the maximum over the three).  Returns 0 if the descriptor is invalid.
 * Size: the sketch and the once-orthonormalised basis as bf16 pairs (8 * n_tokens * rank bytes), the split-K
 * partial sums of V and of the Gram matrices, the sampled rows and the test matrix (4 * rank * d bytes), and,
 * for loract_compress_prenorm without A_out, the normalised input itself.  At n_tokens = 16384, d = 4096,
 * rank = 256 in bf16 that is about 90 MB, 0.67 of X; it is transient (nothing in it is read after the call
 * returns its results) and can be shared by every layer's call that does not overlap another on the GPU. */
size_t loract_workspace_bytes(const loract_desc_t* desc);

/* Algorithm 1, sampling step: the `rank` distinct row indices, uniform without replacement.  The sample is the
 * first `rank` distinct values of the stream c_i = (w_i * n_tokens) >> 32, w_i = word (i mod 4) of the
 * Philox4x32-10 block with key (seed lo, seed hi) and counter (i div 4, 0, call_id lo, call_id hi),
 * in stream order.  idx_dev: device, `rank` int32, written.  ws: device scratch, >= 256 bytes. */
loract_status_t loract_sample_indices(const loract_desc_t* desc, int32_t* idx_dev, void* ws,
                                      size_t ws_bytes, void* stream);

/* Algorithm 1: sample rows, Y = X A_k^T, t = power_iters times { Y = QR, Y = X (X^T Q) }, Y = QR, U = Q,
 * V = Q^T X.  (t = 0 is the setting of the paper's experiments.)
 * X: device, read only.  U (n_tokens x rank), V (rank x d): device, written.  idx_out: device, `rank`
 * int32, written if not NULL.  U has orthonormal columns; U V is the orthogonal projection of X onto
 * range(Y).  The entries of U are not unique (any orthonormal basis of range(Y) is a valid result).
 * The QR step is done through the Gram matrix of the sketch (Y^T Y = L L^T, Q = Y L^-T); it is repeated once on
 * Q when a condition estimate formed on the device says that one round does not reach max|U^T U - I| <= 1e-3
 * (or when a status bit is set): same subspace either way, no host synchronisation, and the choice is a
 * deterministic function of the input. */
loract_status_t loract_compress(const loract_desc_t* desc, const void* X, void* U, void* V,
                                int32_t* idx_out, void* ws, size_t ws_bytes, void* stream);

/* Section 3.1, Reconstruct: X_out = U V (n_tokens x d, row stride ldx, dtype of the descriptor). */
loract_status_t loract_reconstruct(const loract_desc_t* desc, const void* U, const void* V,
                                   void* X_out, void* stream);

/* Section 3.1, the gradient taken at the reconstructed activation, for a linear consumer Z = X W:
 * dW = (U V)^T G, evaluated as V^T (U^T G) so that U V is never formed.  G: device, n_tokens x g, row
 * stride ldg, dtype of the descriptor; several consumers can be served by one call with their
 * gradients concatenated along columns.  1 <= g <= 256.  dW: device, d x g fp32, row stride g; if
 * `accumulate` is non-zero the result is added to dW, otherwise dW is overwritten. */
loract_status_t loract_weight_grad(const loract_desc_t* desc, const void* U, const void* V,
                                   const void* G, int32_t g, int64_t ldg, float* dW, int accumulate,
                                   void* ws, size_t ws_bytes, void* stream);

/* Section 3.3, the pre-norm unit: A = Norm(X) is computed once, compressed once, and that one factor
 * pair serves the Norm backward and every projection inside the sub-layer.
 *   RMS   : A = X * rstd * gamma,           rstd_i = 1 / sqrt(mean_j X_ij^2 + eps)
 *   LAYER : A = (X - mean_i) * rstd_i * gamma + beta   (textbook LayerNorm; beta may be NULL)
 * gamma, beta: device, d elements, dtype of the descriptor.  rstd: device, n_tokens fp32, written.
 * mean: device, n_tokens fp32, written for LAYER (may be NULL for RMS).  A_out: device, n_tokens x d with
 * row stride d, written if not NULL (the forward pass needs it as the sub-layer input); if NULL the
 * normalised matrix lives only in `ws`.  U, V, ws, stream as for loract_compress; (U, V) factor A. */
loract_status_t loract_compress_prenorm(const loract_desc_t* desc, const void* X, const void* gamma,
                                        const void* beta, float eps, int32_t kind, void* A_out,
                                        float* rstd, float* mean, void* U, void* V, int32_t* idx_out,
                                        void* ws, size_t ws_bytes, void* stream);

/* Section 3.3, the backward pass of the pre-norm unit (RMS form) from the compressed normalised activation:
 *   Xbar = A~ / gamma,  grad_Xbar = grad_A * gamma,
 *   grad_X = rstd * (grad_Xbar - Xbar * (1/d) sum_j [grad_Xbar * Xbar]_j),        A~ = U V.
 * (U, V) and rstd are those of loract_compress_prenorm (LORACT_NORM_RMS).  grad_A: device, n_tokens x d, row
 * stride ldx, the gradient with respect to the sub-layer input A (all consumers already summed).  grad_X:
 * device, n_tokens x d, row stride ldx, written.  A~ is never stored: the row means come from the factors
 * ((1/d) U_i . (grad_A V^T)_i, since gamma cancels in the product) and the reconstructed tiles exist only
 * inside the kernel that writes grad_X.  bf16 only (LORACT_ERR_UNSUPPORTED for fp32).  ws: at least
 * loract_prenorm_backward_workspace_bytes(desc) bytes. */
size_t loract_prenorm_backward_workspace_bytes(const loract_desc_t* desc);
loract_status_t loract_prenorm_backward(const loract_desc_t* desc, const void* U, const void* V,
                                        const void* gamma, const float* rstd, const void* grad_A,
                                        void* grad_X, void* ws, size_t ws_bytes, void* stream);

/* Section 3.1, the gradient equation grad_X = grad_Z * dZ/dX taken at the reconstructed activation, for an
 * element-wise Z = f(X) whose saved input A = X was compressed to (U, V):  grad_X = grad_Z * f'(A~), A~ = U V.
 *   LORACT_ACT_SILU : f(a) = a / (1 + exp(-a)),  f'(a) = s (1 + a (1 - s)), s = 1 / (1 + exp(-a))
 *   LORACT_ACT_GELU : f(a) = a Phi(a) (exact form), f'(a) = Phi(a) + a phi(a)
 * grad_Z: device, n_tokens x d, row stride ldx.  grad_X: device, n_tokens x d, row stride ldx, written.  A~ is
 * never stored: its tiles exist only in tensor memory, inside the kernel that writes grad_X (grad_Z is read
 * once, grad_X written once, the factors read once).  bf16 only (LORACT_ERR_UNSUPPORTED for fp32).  Needs no
 * workspace. */
loract_status_t loract_activation_backward(const loract_desc_t* desc, const void* U, const void* V,
                                           const void* grad_Z, int32_t kind, void* grad_X, void* stream);

/* Algorithm 1 (t = 0) on ONE matrix X whose token rows are sharded over several GPUs (sequence or context
 * parallelism), as one joint factorisation: the same U V = P_Y X as loract_compress on the whole X.  Every shard
 * runs the stages below on its own rows [row0, row0 + n_tokens) (desc->n_tokens is the shard's row count, desc->
 * seed / call_id are the same on every shard); between stages the caller adds the small matrices over all shards
 * (an all-reduce with NCCL; what arrives lands in local memory before the next stage reads it) -- the library
 * itself does no communication.  bf16 only; every shard needs at least `rank` rows.
 *   1. loract_joint_sample_rows : the sampling step.  The `rank` sampled rows of the whole matrix (indices in [0, n_global),
 *      the same on every shard); S (rank x d) receives those that live on this shard, zeros elsewhere.
 *      -> add S over the shards (one non-zero contribution per row: exact).
 *   2. loract_joint_sketch      : the sketch.  Y_local = X_local Omega^T with the test matrix Omega made from S_sum (the
 *      same bits on every shard), and W_partial (rank x rank fp32) = Y_local^T Y_local.  -> add W_partial.
 *   3. loract_joint_orthonormalise, round 0 : the QR step, first half.  Y_local <- Y_local L^-T with L L^T = W_sum;
 *      W_next_partial = the new Y_local^T Y_local.  -> add W_next_partial.
 *      round 1 : second half.  U_local (n_tokens x rank) = Y_local L^-T with the factor of the second sum.
 *   4. loract_joint_project     : the projection.  V_partial (rank x d fp32) = U_local^T X_local.  -> add V_partial.
 *   5. loract_joint_finish      : V (rank x d, bf16) = V_sum rounded once.
 * The sketch and the once-orthonormalised sketch stay in `ws` between the stages: the same `ws` (at least
 * loract_joint_workspace_bytes(desc) bytes) must be passed to stages 1 to 4 of one factorisation.  The device
 * status word at the start of `ws` is cleared by stage 1 and collects every later stage's conditions. */
size_t loract_joint_workspace_bytes(const loract_desc_t* desc);
loract_status_t loract_joint_sample_rows(const loract_desc_t* desc, int64_t n_global, int64_t row0,
                                         const void* X_local, void* S, int32_t* idx_out, void* ws, size_t ws_bytes,
                                         void* stream);
loract_status_t loract_joint_sketch(const loract_desc_t* desc, const void* X_local, const void* S_sum,
                                    float* W_partial, void* ws, size_t ws_bytes, void* stream);
loract_status_t loract_joint_orthonormalise(const loract_desc_t* desc, int32_t round, const float* W_sum,
                                            float* W_next_partial, void* U_local, void* ws, size_t ws_bytes,
                                            void* stream);
loract_status_t loract_joint_project(const loract_desc_t* desc, const void* U_local, const void* X_local,
                                     float* V_partial, void* ws, size_t ws_bytes, void* stream);
loract_status_t loract_joint_finish(const loract_desc_t* desc, const float* V_sum, void* V, void* stream);

/* The same result as loract_weight_grad, for callers that cannot allocate device memory and so cannot
 * provide `ws`.  (The paper has no counterpart: this is a property of the library, not of the method.)
 * Typical callers: a backward hook running while the framework's caching allocator is locked or out of
 * memory, a runtime with a memory plan fixed ahead of time, a process in which another component owns
 * cudaMalloc.  The intermediate T = U^T G lives in a fixed 1 MiB array inside the library image, which
 * every GPU that loads the library holds until the process exits.  The call itself allocates nothing: no
 * cudaMalloc, no cudaFree, no allocating library routine.
 *   - Limit: 256 + 2 * (4 * rank * g rounded up to 256) bytes must fit in the 1 MiB, i.e. rank * g <= 131040
 *     (every valid rank <= 512 with g <= 255; rank 512 with g = 256 does not fit).  Beyond it the call
 *     returns LORACT_ERR_UNSUPPORTED and launches nothing.  Other argument rules as loract_weight_grad.
 *   - The first call on each device looks up the array's device address (the device must be current);
 *     make that first call before any stream capture begins.
 *   - All calls share the one array, which keeps the previous call's contents; the call clears what must
 *     start at zero.  Two calls that overlap on the GPU (different streams, or different threads) race
 *     on it: serialise them.
 *   - The device status word of this entry point is the first word of that array; it is not readable
 *     through loract_read_device_status.  loract_weight_grad_static_status copies it to *out_host (a HOST
 *     pointer) and synchronises `stream`; it allocates nothing either.  A non-zero word (an expired wait)
 *     means dW of the last call is not valid. */
loract_status_t loract_weight_grad_static(const loract_desc_t* desc, const void* U, const void* V,
                                          const void* G, int32_t g, int64_t ldg, float* dW, int accumulate,
                                          void* stream);
loract_status_t loract_weight_grad_static_status(uint32_t* out_host, void* stream);

/* Comparator of Section 3.2: randomized SVD at the same rank -- Algorithm 1 with a Gaussian test matrix
 * of rank + oversample columns (Philox + Box-Muller, counter word 1 set to 1) and `power_iters`
 * iterations of Y = X (X^T Q).  Writes the un-truncated pair: Uq (n_tokens x l), B (l x d), l = rank +
 * oversample (a multiple of 8, <= 640; oversample <= 128).  The cut from l to `rank` columns (the singular value decomposition
 * of the small matrix B) is left to the caller.  bf16 only.  ws must hold loract_rsvd_workspace_bytes. */
size_t loract_rsvd_workspace_bytes(const loract_desc_t* desc, int32_t oversample);
loract_status_t loract_rsvd(const loract_desc_t* desc, int32_t oversample, const void* X, void* Uq,
                            void* B, void* ws, size_t ws_bytes, void* stream);

/* Copies the device status word at the start of `ws` to *out_host.  Synchronises `stream`. */
loract_status_t loract_read_device_status(const void* ws, uint32_t* out_host, void* stream);

/* What a device status word means for the call that produced it: LORACT_ERR_TIMEOUT if a bounded wait
 * expired (outputs unspecified), LORACT_ERR_NUMERIC if a non-finite value reached the factorisation or the
 * sampler ran short (outputs written but meaningless), LORACT_OK otherwise (a clamped pivot alone is a
 * warning: the factors are valid).  Pure host function. */
loract_status_t loract_status_from_device_word(uint32_t word);

const char* loract_status_string(loract_status_t s);

/* Number of kernels the library has launched in this process (all entry points); the benchmark
 * reports the difference across its timed region. */
uint64_t loract_kernel_launch_count(void);

#ifdef __cplusplus
}
#endif
#endif /* LORACT_H_ */

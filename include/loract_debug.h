/*
 * loract_debug.h -- test hooks of libloract: the two building blocks every entry point of loract.h is
 * composed of, exported so that the GPU tests can check them in isolation.  Not part of the stable ABI.
 * All pointers are DEVICE pointers owned by the caller unless stated; calls are asynchronous on `stream`.
 */
#ifndef LORACT_DEBUG_H_
#define LORACT_DEBUG_H_

#include "loract.h"

#ifdef __cplusplus
extern "C" {
#endif

/* The contraction behind the sketch and the projection of Algorithm 1 and behind Reconstruct:
 * C (M x N) = sum_{t < n_terms} A_t B_t, contraction length K, fp32 accumulation.
 * a_mn = 0: A_t stored [M][K] (row stride lda); a_mn = 1: stored [K][M].  b_mn = 0: B_t stored [N][K]
 * (row stride ldb); b_mn = 1: stored [K][N].  a_type / b_type: 0 fp32, 1 bf16.  A and B point to
 * n_terms operand pointers each (HOST arrays of device pointers).  out_mode: 0 fp32 into C0, 1 bf16 into
 * C0, 2 bf16 hi/lo pair into C0/C1, 3 fp64 into C0 (CUDA-core kernel only).  splits > 1 writes `splits`
 * partial results `split_stride` elements apart (fp32/fp64 only).  engine: 0 CUDA-core kernel, 1 tensor-core
 * (tcgen05) kernel -- returns LORACT_ERR_UNSUPPORTED if that kernel does not take the shape or types.
 * status_word: device uint32 that receives LORACT_DEV_* bits, may be NULL. */
loract_status_t loract_debug_gemm(int32_t M, int32_t N, int32_t K, int32_t a_mn, int32_t b_mn,
                                  const void* const* A, int64_t lda, const void* const* B, int64_t ldb,
                                  int32_t a_type, int32_t b_type, int32_t n_terms, int32_t out_mode,
                                  void* C0, void* C1, int64_t ldc, int32_t splits, int64_t split_stride,
                                  int32_t acc64, int32_t engine, uint32_t* status_word, void* stream);

/* The same contraction with the sum of the terms before `halve_at_term` multiplied by 1/2 before that term's
 * products are added: C = (A_0 B_0 + ... ) / 2 + A_h B_h + ...  (0: the plain sum; must be < n_terms).  The tall Gram
 * products of the orthonormalisation use it with {Yl^T Yl, Yh^T Yh, Yh^T Yl} and h = 2. */
loract_status_t loract_debug_gemm_halved(int32_t M, int32_t N, int32_t K, int32_t a_mn, int32_t b_mn,
                                         const void* const* A, int64_t lda, const void* const* B, int64_t ldb,
                                         int32_t a_type, int32_t b_type, int32_t n_terms, int32_t halve_at_term,
                                         int32_t out_mode, void* C0, void* C1, int64_t ldc, int32_t splits,
                                         int64_t split_stride, int32_t acc64, int32_t engine, uint32_t* status_word,
                                         void* stream);

/* out (r x r, fp32, device) = S + S^T, S the sum in index order of `n_partials` r x r fp32 matrices `stride` elements
 * apart: the step that turns the partial sums of the halved-accumulator Gram product into the symmetric Gram matrix. */
loract_status_t loract_debug_reduce_sym(const float* partials, int32_t n_partials, int64_t stride, int32_t r,
                                        float* out, void* stream);

/* The projection step of Algorithm 1 alone, exactly as loract_compress runs it (same kernels, same launch shapes):
 * V (rank x d) = U^T X from a stored U (n_tokens x rank).  ws as for loract_compress.  For timing that step in
 * isolation. */
loract_status_t loract_debug_project(const loract_desc_t* desc, const void* U, const void* X, void* V, void* ws,
                                     size_t ws_bytes, void* stream);

/* The tensor-core kernel exists in two forms: one CTA per 128-row tile, and a pair of CTAs (tcgen05
 * cta_group::2) per 256-row tile, chosen by shape.  on = 0 keeps every contraction on the one-CTA form, so
 * that a test can compare the two; on = 1 (the default) restores the choice by shape.  Process-wide. */
void loract_debug_set_pair_mode(int32_t on);

/* The orthonormalisation of the bf16 path runs its second Gram round only when the first round's Gram matrix W
 * was not conditioned well enough for one: a one-CTA kernel forms est = trace((D W D)^-1), D = diag(W)^(-1/2),
 * from the inverse factor and compares est times the number of 64-row blocks per accumulation chain of the Gram
 * product with a threshold (widths up to 512; above that both rounds always run).
 * This sets the threshold, process-wide: a negative value forces both rounds, +infinity allows one round whenever
 * no status bit is set, 0 restores the default.  After a call the status block at the head of the workspace
 * holds, as 32-bit words 4, 5, 6: whether the second round ran (0 / 1), est (float bits), the number of rounds. */
void loract_debug_set_round_gate(float threshold);

/* The deciding kernel alone.  W: r x r fp32 (device, leading dimension r), linv_hi: r x r bf16 lower triangular
 * (device), r a multiple of 8 up to 640; status_word: device uint32 or NULL.  words (device, 3 x uint32) receives
 * { est > threshold or est not finite or *status_word != 0,  est = sum_ij linv_ij^2 W_jj as float bits,
 *   1 or 2 = the number of rounds }. */
loract_status_t loract_debug_round_gate(const float* W, const void* linv_hi, int32_t r, float threshold,
                                        const uint32_t* status_word, uint32_t* words, void* stream);

/* Stage trace.  Between trace_begin and trace_end every kernel the library launches on `stream` is followed by
 * a CUDA event; trace_end synchronises the stream and writes, per kernel in launch order, a label (64 bytes
 * each, zero-terminated: the step of the path and the kernel's launch function) and the time from the
 * previous event to this kernel's event in microseconds.  Returns the number of entries (at most max_entries),
 * or -1.  The events keep neighbouring kernels from overlapping, so the sum is a little above the untraced
 * time.  One trace at a time, from one host thread. */
void loract_debug_trace_begin(void* stream);
int32_t loract_debug_trace_end(void* stream, char* names, float* micros, int32_t max_entries);

/* The give-up path of the bounded device-side waits, exercised without a fault: launches one tiny kernel in
 * which a thread waits on a barrier that nothing ever completes, using the same wait helper as the tensor-core
 * engine (which = 0) or as the cluster factorisation kernel (which = 1, a cluster of two CTAs), with
 * `limit_ns` (1 ns to 100 ms) in place of the built-in limit.  The wait gives up, the kernel ORs
 * LORACT_DEV_WAIT_EXPIRED into *status_word (device uint32) and returns; the context stays usable. */
loract_status_t loract_debug_wait_expiry(int32_t which, uint64_t limit_ns, uint32_t* status_word, void* stream);

/* The cudaError_t behind the most recent LORACT_ERR_CUDA returned by any entry point (0 if none yet). */
int32_t loract_debug_last_cuda_error(void);

/* The small-block step of the orthonormalisation (the QR step of Algorithm 1 done through Gram matrices):
 * W = sum of n_partials r x r matrices (fp32 if partial_f64 == 0, else fp64; `partial_stride` elements
 * apart); L L^T = W + shift_rel * mean(diag W) * I; writes L^{-1} (lower triangular, row-major) as fp32
 * (linv_f32), as a bf16 hi/lo pair (linv_hi, linv_lo), any of which may be NULL.  use_f64 selects the
 * arithmetic.  scratch: 2*r*r + 2*256*(256 + max(r-256,0) + max(r-512,0)) elements of the compute type.  r a multiple of 8, <= 640. */
loract_status_t loract_debug_small_block(int32_t r, const void* partials, int32_t partial_f64,
                                         int32_t n_partials, int64_t partial_stride, int32_t use_f64,
                                         float shift_rel, void* scratch, float* linv_f32, void* linv_hi,
                                         void* linv_lo, uint32_t* status_word, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* LORACT_DEBUG_H_ */

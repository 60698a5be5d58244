// Internal declarations shared by the translation units of libloract (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/loract.h"

namespace loract {

// ---------------------------------------------------------------- launch accounting
// Called after every kernel launch: counts it and, while a trace is open (test hook), records an event
// behind it on `stream` under the label set with trace_label().
void count_launch(const char* kernel = "", cudaStream_t stream = nullptr);
void trace_label(const char* label);

// The argument rules every entry point shares (include/loract.h, "Conventions"): LORACT_OK or the error.
loract_status_t check_desc(const loract_desc_t* d);

#define LORACT_CUDA_TRY(expr)                          \
  do {                                                 \
    cudaError_t _e = (expr);                           \
    if (_e != cudaSuccess) return _e;                  \
  } while (0)

// ---------------------------------------------------------------- programmatic dependent launch
// The kernels of one call run back to back on one stream.  Launched with programmatic stream
// serialisation, a kernel may start (be scheduled, set up shared memory, barriers, tensor memory) while
// its predecessor is still running; it must then execute pdl_wait() before its first access to global
// memory, which returns once the predecessor has completed and its writes are visible.
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename Kern, typename... Args>
cudaError_t launch_pdl(Kern kernel, dim3 grid, dim3 block, size_t smem, cudaStream_t stream, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}
#endif

// ---------------------------------------------------------------- generic contraction
// C (M x N) = sum over terms of  A_t (M x K) * B_t (K x N), fp32 (or fp64) accumulation.
// Operands are row-major arrays; a_mn / b_mn say which index is contiguous in memory:
//   a_mn == false : A stored as [M][K]  (K-major)      a_mn == true : A stored as [K][M]  (M-major)
//   b_mn == false : B stored as [N][K]  (K-major)      b_mn == true : B stored as [K][N]  (N-major)
// Several terms share shapes and leading dimensions; they exist for split-precision products
// (x = hi + lo in bf16: hi*hi + hi*lo + lo*hi).
enum OutMode : int {
  OUT_F32 = 0,    // C0: float
  OUT_BF16 = 1,   // C0: bf16
  OUT_SPLIT = 2,  // C0: bf16 hi, C1: bf16 lo  (hi = bf16(x), lo = bf16(x - hi))
  OUT_F64 = 3,    // C0: double (SIMT path only)
  // C0: bf16, C0[m][n] = row_a[m] * col[n] * E[m][n] - row_b[m] / col[n] * acc[m][n]  (tensor-core path only):
  // the input gradient of the RMS pre-norm unit from a reconstructed tile that is never stored
  OUT_RMS_BWD = 4,
  // C0: bf16, C0[m][n] = E[m][n] * f'(acc[m][n]), f = SiLU (ep_kind 0) or GELU (ep_kind 1)  (tensor-core path
  // only): the input gradient of an element-wise activation from a reconstructed tile that is never stored
  OUT_ACT_BWD = 5
};

enum ElemType : int { ELEM_F32 = 0, ELEM_BF16 = 1, ELEM_F64 = 2 };

struct GemmTerm {
  const void* A;
  const void* B;
};

struct GemmDesc {
  int M = 0, N = 0, K = 0;
  bool a_mn = false, b_mn = false;
  int64_t lda = 0, ldb = 0;  // leading dimension (elements) of the stored arrays
  int a_type = ELEM_BF16, b_type = ELEM_BF16;
  int n_terms = 1;
  GemmTerm terms[4];
  int out = OUT_F32;
  void* C0 = nullptr;
  void* C1 = nullptr;
  int64_t ldc = 0;
  // split over K: split s handles a contiguous K range and writes C0 + s * split_stride (fp32/f64 out)
  int splits = 1;
  int64_t split_stride = 0;
  bool acc64 = false;      // SIMT path: accumulate in double
  bool accumulate = false; // SIMT path, OUT_F32, splits == 1: C += result
  float alpha = 1.0f;      // SIMT path: C = alpha * sum
  // OUT_RMS_BWD: E (bf16, M x N, leading dimension ep_ld), per-row and per-column coefficients
  const void* ep_E = nullptr;
  int64_t ep_ld = 0;
  const float* ep_row_a = nullptr;
  const float* ep_row_b = nullptr;
  const void* ep_col = nullptr;
  int ep_kind = 0;         // OUT_ACT_BWD: which activation
  // Two-CTA kernel, K-major A: loads of A from this K element on ask L2 to evict them last (a later kernel
  // reads the same bytes again); negative: no hint.
  int64_t a_keep_from_k = -1;
  // The sum of the terms before this one is multiplied by 1/2 before this term's products are added
  // (result = (t_0 + ... + t_{h-1}) / 2 + t_h + ...); 0 or negative: plain sum.  With the pair {A^T A, A^T B} and
  // h = 1 the result D gives D + D^T = A^T A + A^T B + B^T A: a symmetric three-term sum for two terms' work.
  int halve_at_term = 0;
  // Tensor-core path: a device word written by a kernel at least TWO launches earlier in the same stream (the gated
  // kernel reads it before its griddepcontrol.wait); when it is zero the launch does nothing (no loads, no products,
  // C untouched).  nullptr: unconditional.
  const uint32_t* gate = nullptr;
  // Tensor-core path: the launch stores zero into the status word before any of its waits can set a bit in it (the
  // first kernel of a call clears the word itself instead of a memset in front of it).
  // fp32 32 x 32 tile kernel (gemm_f32_small_launch): optional bf16 hi / lo copies of the result (leading dimension ldc)
  void* split_hi = nullptr;
  void* split_lo = nullptr;
  bool clear_status = false;
  // Tensor-core path, OUT_SPLIT: a device word written by an earlier kernel; when it is zero only C0 (the leading bf16
  // part) is written and C1 keeps its old contents.
  const uint32_t* lo_gate = nullptr;
};

// tcgen05 engine: bf16 operands, fp32 accumulation in tensor memory.  Returns cudaErrorNotSupported
// for shapes it does not take (the caller then uses the SIMT kernel).
bool gemm_tc_supported(const GemmDesc& g);
cudaError_t gemm_tc_launch(const GemmDesc& g, uint32_t* dev_status, cudaStream_t stream);
int gemm_tc_pick_splits(int M, int N, int K, bool a_mn, bool b_mn, int max_splits = 32);
void gemm_tc_set_pair_mode(int on);   // test hook: 0 keeps every contraction on the one-CTA kernel
// Test hooks for the give-up path of the bounded waits: a kernel that waits (with the engine's / the cluster
// kernel's own wait) on a barrier nothing completes, for at most limit_ns, then sets LORACT_DEV_WAIT_EXPIRED.
cudaError_t gemm_tc_wait_probe_launch(uint32_t* dev_status, uint64_t limit_ns, cudaStream_t stream);
cudaError_t small_block_cluster_wait_probe_launch(uint32_t* dev_status, uint64_t limit_ns, cudaStream_t stream);

// Plain CUDA-core kernel for any shape and type (fp32 path, small or odd shapes).
cudaError_t gemm_simt_launch(const GemmDesc& g, cudaStream_t stream);
// fp32 x fp32 -> fp32 for matrices of a few hundred rows and columns (32 x 32 tiles, one per CTA).
// `second`: an independent product carried by the same launch (both may read what earlier launches wrote;
// neither may read the other's output).
cudaError_t gemm_f32_small_launch(const GemmDesc& g, cudaStream_t stream, const GemmDesc* second = nullptr);

// ---------------------------------------------------------------- sampler and gather
// idx_copy (optional) receives the same indices; clear_status: the kernel sets the status word instead of OR-ing
// into it (for the first kernel of a call).
cudaError_t sample_indices_launch(uint64_t seed, uint64_t call_id, uint32_t n_rows, int rank,
                                  int32_t* idx_dev, uint32_t* dev_status, cudaStream_t stream,
                                  int32_t* idx_copy = nullptr, bool clear_status = false);
// dst (rank x d, stride d) = src[idx, :] (stride ld); 16-byte loads.  elem_bytes 2 or 4.
cudaError_t gather_rows_launch(const void* src, int64_t ld, const int32_t* idx, int rank, int64_t d,
                               int elem_bytes, void* dst, cudaStream_t stream);
// The same for one shard of a token-sharded matrix (src = rows [row0, row0 + n_local) of the whole matrix, idx in
// whole-matrix row numbers): rows that live on another shard are written as zeros.
cudaError_t gather_rows_window_launch(const void* src, int64_t ld, const int32_t* idx, int rank, int64_t d,
                                      int elem_bytes, int64_t row0, int64_t n_local, void* dst, cudaStream_t stream);
// Gaussian test matrix for the RSVD comparator: dst (l x d bf16, row-major) with
// dst[c][j] = z(j * l + c), z the Philox + Box-Muller stream (counter word 1 = 1).
cudaError_t gaussian_rows_launch(uint64_t seed, uint64_t call_id, int l, int64_t d,
                                 __nv_bfloat16* dst, cudaStream_t stream);

// ---------------------------------------------------------------- small-block factorisation
// From the symmetric positive semi-definite r x r matrix  W = sum_s P_s  (P_s fp32 or fp64, row-major,
// stride r, consecutive partials `partial_stride` elements apart) computes the inverse of the
// Cholesky factor of  W + shift_rel * mean(diag W) * I :  Linv = L^{-1} (lower triangular), so that
// (Y Linv^T) has orthonormal columns when W = Y^T Y.  Outputs (any may be null): Linv as an fp32 or
// fp64 matrix, and as a bf16 hi/lo pair.  `scratch` holds r*r + 1024*ceil(r/32) elements of the compute type.
struct SmallBlockArgs {
  int r = 0;
  const void* partials = nullptr;
  int partial_type = ELEM_F32;
  int n_partials = 1;
  int64_t partial_stride = 0;
  bool use_f64 = false;  // compute type
  void* scratch = nullptr;
  float shift_rel = 0.f;
  // shared-memory cluster kernel and the block scheme built on it: each diagonal entry is also multiplied by
  // (1 + shift_diag_rel), a shift relative to the entry itself (the scale-invariant form, which leaves a
  // matrix whose diagonal spans several orders of magnitude as well conditioned as its scaled form)
  float shift_diag_rel = 0.f;
  // device word written by an earlier kernel of the stream; zero: the launch does nothing.  nullptr: unconditional.
  const uint32_t* gate = nullptr;
  // shared-memory cluster kernel only (r <= 256): three words that receive what round_gate_launch would write for
  // this matrix and its inverse factor, computed inside the factorisation (no extra launch)
  uint32_t* gate_out = nullptr;
  float gate_threshold = 0.f;
  void* linv_full = nullptr;  // fp32 (use_f64 == false) or fp64 (use_f64 == true), r x r
  float* linv_f32 = nullptr;  // fp32 copy, r x r
  __nv_bfloat16* linv_hi = nullptr;
  __nv_bfloat16* linv_lo = nullptr;
  uint32_t* dev_status = nullptr;
  // row strides (elements) of the partial matrices and of the outputs; 0 means r.  The matrix may be a
  // diagonal sub-block of a larger one (the r > 256 path factors a 512 x 512 matrix through its 256 x 256 blocks)
  int64_t in_ld = 0, out_ld = 0;
  // Where the scale of the shift and of the pivot floor comes from: by default the mean of the matrix's own
  // diagonal.  A Schur complement that is handed in as "the matrix" can be all rounding noise, so the two-level
  // path points this at the diagonal of the block it was taken from (scale_n entries, stride scale_ld + 1).
  const float* scale_diag = nullptr;
  int scale_n = 0;
  int64_t scale_ld = 0;
};
cudaError_t small_block_launch(const SmallBlockArgs& a, cudaStream_t stream);
// The same computation for r <= 256 in fp32 from fp32 partials, entirely in the shared memory of a
// cluster of eight CTAs (no scratch).  small_block_launch uses it whenever it applies.
bool small_block_cluster_supported(const SmallBlockArgs& a);
cudaError_t small_block_cluster_launch(const SmallBlockArgs& a, cudaStream_t stream);

// ---------------------------------------------------------------- elementwise helpers
// out = sum_s partials[s] (fixed order), written as fp32 and/or bf16.
// X21 of a 2 x 2 block lower-triangular inverse as bf16 hi/lo (and optionally fp32), plus zeros in the block
// above the diagonal: src (rows x cols fp32, leading dimension ld) -> hi/lo at the same place.
cudaError_t split_block_launch(const float* src, int rows, int cols, int64_t ld, __nv_bfloat16* hi,
                               __nv_bfloat16* lo, cudaStream_t stream, const uint32_t* gate = nullptr);
// Zero fill of up to three ranges (16-byte aligned, sizes multiples of 16; a null range has size 0), one launch.
// Optionally the same launch also forms sum_dst[i] = sum over n_src partials of sum_src[q * src_stride + i], i < count.
cudaError_t zero3_gated_launch(void* a, size_t a_bytes, void* b, size_t b_bytes, void* c, size_t c_bytes,
                               const uint32_t* gate, cudaStream_t stream, const float* sum_src = nullptr,
                               int n_src = 0, int64_t src_stride = 0, int64_t count = 0, float* sum_dst = nullptr);
cudaError_t reduce_partials_launch(const float* partials, int n_partials, int64_t stride,
                                   int64_t count, float* out_f32, __nv_bfloat16* out_bf16,
                                   cudaStream_t stream, const uint32_t* gate = nullptr);
// out (r x r) = S + S^T, S the fixed-order sum of the partials (each r x r, leading dimension r).
// gate (optional): device word; zero means the launch does nothing.
cudaError_t reduce_sym_launch(const float* partials, int n_partials, int64_t stride, int r, float* out,
                              cudaStream_t stream, const uint32_t* gate = nullptr);
// After the first orthonormalisation round: decides on the device whether the second round is needed.
// W (r x r fp32, leading dimension r) is the Gram matrix that was factored, linv_hi the leading bf16 part of the
// inverse factor L^-1 (leading dimension r).  With D = diag(W)^(-1/2) the kernel forms
//   est = sum_ij (L^-1)_ij^2 W_jj = trace((D W D)^-1),
// which lies between 1 / lambda_min and r / lambda_min of the diagonally scaled Gram matrix, the quantity that
// multiplies the rounding error of W in the orthogonality defect of Y L^-T.  gate_words[0] = 1 if est > threshold, est is
// not finite, or the status word is non-zero (a clamped pivot, a non-finite input), else 0; gate_words[1] = est
// (float bits); gate_words[2] = rounds that will run (1 or 2).  One cluster of eight CTAs, fixed summation order.
cudaError_t round_gate_launch(const float* W, const __nv_bfloat16* linv_hi, int r, float threshold,
                              const uint32_t* dev_status, uint32_t* gate_words, cudaStream_t stream);
// dst = src (count bf16 elements, both 16-byte aligned, count a multiple of 8) when *gate != 0; nothing otherwise.
cudaError_t copy_bf16_gated_launch(const __nv_bfloat16* src, __nv_bfloat16* dst, int64_t count, const uint32_t* gate,
                                   cudaStream_t stream);
// out = sum_s partials[s] as a bf16 triple hi + mid + lo (rows x cols, leading dimensions ld_in / ld_out).
cudaError_t reduce_split3_launch(const float* partials, int n_partials, int64_t stride, int rows, int cols,
                                 int64_t ld_in, int64_t ld_out, __nv_bfloat16* hi, __nv_bfloat16* mid,
                                 __nv_bfloat16* lo, cudaStream_t stream);
// Section 3.3 backward, row coefficients: inner_i = (1 / d) sum_k U[i][k] P[i][k] (P = grad_A V^T, fp32, n x r),
// row_a[i] = rstd[i], row_b[i] = rstd[i] * inner_i.  One warp per row.
cudaError_t rms_backward_rows_launch(const __nv_bfloat16* U, const float* P, const float* rstd, int64_t n, int r,
                                     int64_t d, float* row_a, float* row_b, cudaStream_t stream);
// Section 3.3 forward: A = Norm(X); per-row rstd (and mean for LayerNorm).  One warp per row.
cudaError_t norm_forward_launch(const void* X, int64_t n, int64_t d, int64_t ldx, int elem_type,
                                const void* gamma, const void* beta, float eps, int kind, void* A,
                                int64_t lda, float* rstd, float* mean, cudaStream_t stream);

}  // namespace loract

// Orthonormalisation of the small (r x r) blocks of the decomposition: Cholesky factor of a Gram
// matrix and the inverse of that factor, in one thread-block-cluster kernel.
//
// Algorithm 1 orthonormalises the tall sketch Y (its QR step, Y = QR).  Here that is done through Gram
// matrices: with W = Y^T Y = L L^T, Q = Y L^{-T} has orthonormal columns.  The only serial work is on
// the r x r matrix W, r <= 512, and this kernel does it: left-looking blocked Cholesky with panels of
// 32 columns (the 32 x 32 diagonal block is factored by one warp in registers with shuffles, the
// panel below it is a product with the inverse of that block), then the inverse of L by block
// forward substitution, one 32-column block per CTA at a time, kept in shared memory.  The CTAs of the
// cluster split the rows of every panel and synchronise with the hardware cluster barrier.
#include <cooperative_groups.h>

#include <atomic>

#include "common.cuh"

namespace cg = cooperative_groups;

namespace loract {

namespace {

constexpr int kNB = 32;             // panel width
constexpr int kSBThreads = 512;     // 16 warps per CTA
constexpr int kSBWarps = kSBThreads / 32;
constexpr int kCluster = 8;

struct SBParams {
  int r;
  const void* partials;
  int partial_is_f64;
  int n_partials;
  int64_t partial_stride;
  void* scratch;       // T[r*r] (W, then L in its lower triangle) + T[1024*ceil(r/32)] (inverses of diagonal blocks)
  float shift_rel;
  void* linv_full;     // T, r x r, or null
  float* linv_f32;
  __nv_bfloat16* linv_hi;
  __nv_bfloat16* linv_lo;
  uint32_t* dev_status;
};

template <typename T> __device__ __forceinline__ T ldcg_t(const T* p) { return __ldcg(p); }

template <typename T> __device__ __forceinline__ T rsqrt_t(T x);
template <> __device__ __forceinline__ float rsqrt_t<float>(float x) { return rsqrtf(x); }
template <> __device__ __forceinline__ double rsqrt_t<double>(double x) { return 1.0 / sqrt(x); }

template <typename T>
__device__ __forceinline__ T read_partial_sum(const SBParams& p, int i, int j) {
  T s = (T)0;
  const int64_t off = (int64_t)i * p.r + j;
  if (p.partial_is_f64) {
    const double* q = (const double*)p.partials;
    for (int k = 0; k < p.n_partials; ++k) s += (T)__ldg(q + (int64_t)k * p.partial_stride + off);
  } else {
    const float* q = (const float*)p.partials;
    for (int k = 0; k < p.n_partials; ++k) s += (T)__ldg(q + (int64_t)k * p.partial_stride + off);
  }
  return s;
}

template <typename T>
__global__ void __cluster_dims__(kCluster, 1, 1) __launch_bounds__(kSBThreads)
small_block_kernel(SBParams p) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  cg::cluster_group cluster = cg::this_cluster();
  const int n_cta = (int)cluster.num_blocks();
  const int cta = (int)cluster.block_rank();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = p.r;
  const int n_blk = (r + kNB - 1) / kNB;
  T* W = (T*)p.scratch;
  T* Dinv = W + (int64_t)r * r;  // n_blk blocks of 32 x 32, block b at Dinv + b * 1024

  // shared memory carve-up
  T* big = (T*)smem_raw;                       // LrowT (c x 32) during the factorisation, Xs afterwards
  T* dinv_s = big + (int64_t)r * kNB;          // 32 x 33
  T* sblk = dinv_s + kNB * (kNB + 1);          // 32 x 32
  __shared__ T s_red[kSBWarps];
  __shared__ T s_shift, s_floor;

  // ---- phase 0: W = sym(sum of partials) + shift I (lower triangle only)
  {
    T t = (T)0;
    for (int i = tid; i < r; i += kSBThreads) t += read_partial_sum<T>(p, i, i);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) s_red[warp] = t;
    __syncthreads();
    if (tid == 0) {
      T tr = (T)0;
      for (int q = 0; q < kSBWarps; ++q) tr += s_red[q];
      T mean_diag = tr / (T)r;
      if (!(mean_diag == mean_diag) || mean_diag > (T)3.0e38 || mean_diag < (T)0) {
        if (p.dev_status && cta == 0) atomicOr(p.dev_status, LORACT_DEV_NONFINITE);
        mean_diag = (T)1;
      }
      if (mean_diag == (T)0) mean_diag = (T)1;
      s_shift = (T)p.shift_rel * mean_diag;
      s_floor = mean_diag * (sizeof(T) == 8 ? (T)1e-15 : (T)1e-7);
    }
    __syncthreads();
  }
  const T shift = s_shift, pivot_floor = s_floor;
  {
    const int64_t total = (int64_t)r * r;
    for (int64_t e = (int64_t)cta * kSBThreads + tid; e < total; e += (int64_t)n_cta * kSBThreads) {
      const int i = (int)(e / r), j = (int)(e - (int64_t)i * r);
      if (j > i) continue;
      T v = (T)0.5 * (read_partial_sum<T>(p, i, j) + read_partial_sum<T>(p, j, i));
      if (i == j) v += shift;
      W[e] = v;
    }
  }
  __threadfence();
  cluster.sync();

  // ---- blocked left-looking Cholesky
  for (int b = 0; b < n_blk; ++b) {
    const int J0 = b * kNB;
    const int nbw = min(kNB, r - J0);
    // (A) panel <- panel - L[:, :J0] L[J0:J0+nbw, :J0]^T for rows >= J0
    if (J0 > 0) {
      for (int e = tid; e < J0 * kNB; e += kSBThreads) {
        const int c = e / kNB, jj = e - c * kNB;
        big[e] = (jj < nbw) ? ldcg_t(W + (int64_t)(J0 + jj) * r + c) : (T)0;
      }
      __syncthreads();
      for (int i = J0 + cta * kSBWarps + warp; i < r; i += n_cta * kSBWarps) {
        T acc = (lane < nbw) ? ldcg_t(W + (int64_t)i * r + J0 + lane) : (T)0;
        for (int c0 = 0; c0 < J0; c0 += 32) {
          const T v = ldcg_t(W + (int64_t)i * r + c0 + lane);
#pragma unroll
          for (int q = 0; q < 32; ++q) acc -= __shfl_sync(0xffffffffu, v, q) * big[(c0 + q) * kNB + lane];
        }
        if (lane < nbw) W[(int64_t)i * r + J0 + lane] = acc;
      }
      __threadfence();
      cluster.sync();
    }
    // (B) every CTA factors the diagonal block redundantly (warp 0, one row per lane, in registers)
    if (warp == 0) {
      T a[kNB];
#pragma unroll
      for (int j = 0; j < kNB; ++j) {
        T v = (lane == j) ? (T)1 : (T)0;
        if (lane < nbw && j <= lane && j < nbw) v = ldcg_t(W + (int64_t)(J0 + lane) * r + J0 + j);
        a[j] = v;
      }
      bool clamped = false;
#pragma unroll
      for (int k = 0; k < kNB; ++k) {
        T akk = __shfl_sync(0xffffffffu, a[k], k);
        // a pivot that is not safely positive is replaced by the floor and its column is dropped
        const bool bad = !(akk > pivot_floor);
        if (bad) { akk = pivot_floor; clamped = true; }
        const T rinv = rsqrt_t<T>(akk);
        const T lik = (lane == k) ? akk * rinv : ((lane > k && !bad) ? a[k] * rinv : (T)0);
        a[k] = lik;
#pragma unroll
        for (int j = k + 1; j < kNB; ++j) {
          const T ljk = __shfl_sync(0xffffffffu, lik, j);
          a[j] -= lik * ljk;
        }
      }
      // inverse of the lower-triangular block: lane j solves L x = e_j (column j of the inverse)
      T x[kNB];
#pragma unroll
      for (int i = 0; i < kNB; ++i) {
        T s = (lane == i) ? (T)1 : (T)0;
#pragma unroll
        for (int q = 0; q < i; ++q) s -= __shfl_sync(0xffffffffu, a[q], i) * x[q];
        const T lii = __shfl_sync(0xffffffffu, a[i], i);
        x[i] = (i >= lane) ? s / lii : (T)0;
      }
#pragma unroll
      for (int i = 0; i < kNB; ++i) dinv_s[i * (kNB + 1) + lane] = x[i];  // dinv_s[i][j], lane = j
      // The factored diagonal block itself is never read again (later panels and the inverse use
      // only its inverse), so it is not written back: other CTAs may still be loading the block.
      if (cta == 0) {
#pragma unroll
        for (int i = 0; i < kNB; ++i) Dinv[b * kNB * kNB + i * kNB + lane] = x[i];
        if (clamped && lane == 0 && p.dev_status) atomicOr(p.dev_status, LORACT_DEV_PIVOT_CLAMPED);
      }
    }
    __syncthreads();
    // rows below the diagonal block: L[i, J] = panel[i, :] * inverse(L_JJ)^T
    for (int i = J0 + nbw + cta * kSBWarps + warp; i < r; i += n_cta * kSBWarps) {
      const T v = (lane < nbw) ? ldcg_t(W + (int64_t)i * r + J0 + lane) : (T)0;
      T acc = (T)0;
#pragma unroll
      for (int q = 0; q < kNB; ++q) acc += __shfl_sync(0xffffffffu, v, q) * dinv_s[lane * (kNB + 1) + q];
      if (lane < nbw) W[(int64_t)i * r + J0 + lane] = acc;
    }
    __threadfence();
    cluster.sync();
  }

  // ---- inverse of L by block forward substitution; one 32-column block at a time per CTA
  T* Xs = big;  // Xs[(c - J0) * 32 + jj] = Linv[c][J0 + jj]
  for (int round = 0; round * n_cta < n_blk; ++round) {
    // serpentine order balances the long early blocks against the short late ones
    const int jb = round * n_cta + ((round & 1) ? (n_cta - 1 - cta) : cta);
    if (jb >= n_blk) continue;
    const int J0 = jb * kNB;
    const int nbw = min(kNB, r - J0);
    __syncthreads();
    for (int e = tid; e < kNB * kNB; e += kSBThreads)
      Xs[e] = ldcg_t(Dinv + jb * kNB * kNB + e);
    __syncthreads();
    for (int ib = jb + 1; ib < n_blk; ++ib) {
      const int I0 = ib * kNB;
      const int nrows = min(kNB, r - I0);
      for (int e = tid; e < kNB * kNB; e += kSBThreads) {
        const int i = e / kNB, j = e - i * kNB;
        dinv_s[i * (kNB + 1) + j] = ldcg_t(Dinv + ib * kNB * kNB + e);
      }
      for (int ii = warp; ii < kNB; ii += kSBWarps) {
        T acc = (T)0;
        if (ii < nrows) {
          const int i = I0 + ii;
          for (int c0 = J0; c0 < I0; c0 += 32) {
            const T v = ldcg_t(W + (int64_t)i * r + c0 + lane);
#pragma unroll
            for (int q = 0; q < 32; ++q)
              acc += __shfl_sync(0xffffffffu, v, q) * Xs[(c0 - J0 + q) * kNB + lane];
          }
        }
        sblk[ii * kNB + lane] = acc;
      }
      __syncthreads();
      for (int ii = warp; ii < kNB; ii += kSBWarps) {
        T acc = (T)0;
        for (int q = 0; q <= ii; ++q) acc -= dinv_s[ii * (kNB + 1) + q] * sblk[q * kNB + lane];
        Xs[(I0 - J0 + ii) * kNB + lane] = (ii < nrows) ? acc : (T)0;
      }
      __syncthreads();
    }
    // write the column block (zeros above the diagonal block)
    for (int64_t e = tid; e < (int64_t)r * kNB; e += kSBThreads) {
      const int i = (int)(e / kNB), jj = (int)(e - (int64_t)i * kNB);
      if (jj >= nbw) continue;
      const T v = (i >= J0) ? Xs[(i - J0) * kNB + jj] : (T)0;
      const int64_t off = (int64_t)i * r + J0 + jj;
      if (p.linv_full) ((T*)p.linv_full)[off] = v;
      const float f = (float)v;
      if (p.linv_f32) p.linv_f32[off] = f;
      if (p.linv_hi) {
        const __nv_bfloat16 hi = __float2bfloat16(f);
        p.linv_hi[off] = hi;
        if (p.linv_lo) p.linv_lo[off] = __float2bfloat16(f - __bfloat162float(hi));
      }
    }
  }
  cluster.sync();  // no CTA of the cluster exits while others may still read its results' inputs
}

template <typename T>
cudaError_t launch_typed(const SBParams& p, cudaStream_t stream) {
  const size_t smem = ((size_t)p.r * kNB + kNB * (kNB + 1) + kNB * kNB) * sizeof(T);
  static std::atomic<bool> configured[64];  // per device and instantiation, zero-initialised
  int dev = 0;
  LORACT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    LORACT_CUDA_TRY(cudaFuncSetAttribute(small_block_kernel<T>,
                                         cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  small_block_kernel<T><<<kCluster, kSBThreads, smem, stream>>>(p);
  count_launch(__func__, stream);
  return cudaGetLastError();
}

}  // namespace

// r > 256 in fp32: the matrix as 2 x 2 blocks, W = [W11 . ; W21 W22], the leading block 256 wide.
//   L11 = chol(W11), X11 = L11^-1            (shared-memory cluster kernel)
//   L21 = W21 X11^T,  S = W22 - L21 L21^T    (fp32 CUDA-core products)
//   L22 = chol(S), X22 = L22^-1              (the same again if S is wider than 256, else the cluster kernel)
//   X21 = -X22 (L21 X11)                     (fp32 CUDA-core products)
// W (n x n, leading dimension ld) is overwritten by the Schur complements; X (fp32) and the bf16 pair receive the
// inverse factor at the same place and leading dimension.  T: 2 * 256 * (n - 256) floats for this level's two
// temporaries, followed by what the levels below need.  The shift and the pivot floor of every level come from
// the diagonal of the whole matrix's leading block (`scale`): a Schur complement may be nothing but rounding noise.
struct TwoLevelCtx {
  float shift_rel;
  float shift_diag_rel;
  const uint32_t* gate;
  uint32_t* dev_status;
  int64_t ld;
  const float* scale_diag;
  int scale_n;
  cudaStream_t stream;
};

cudaError_t factor_blocks(const TwoLevelCtx& c, float* W, float* X, __nv_bfloat16* hi, __nv_bfloat16* lo, int n,
                          float* T, bool top) {
  const int64_t ld = c.ld;
  if (n <= 256) {
    SmallBlockArgs s;
    s.r = n; s.partials = W; s.partial_type = ELEM_F32; s.n_partials = 1; s.partial_stride = 0;
    s.use_f64 = false; s.shift_rel = c.shift_rel; s.shift_diag_rel = c.shift_diag_rel; s.in_ld = ld; s.out_ld = ld;
    s.linv_f32 = X; s.linv_hi = hi; s.linv_lo = lo; s.dev_status = c.dev_status; s.gate = c.gate;
    if (!top) { s.scale_diag = c.scale_diag; s.scale_n = c.scale_n; s.scale_ld = ld; }
    return small_block_cluster_launch(s, c.stream);
  }
  const int r1 = 256, r2 = n - r1;
  float* T1 = T;
  float* T2 = T1 + (size_t)r2 * r1;
  float* Tnext = T2 + (size_t)r2 * r1;
  LORACT_CUDA_TRY(factor_blocks(c, W, X, hi, lo, r1, Tnext, top));
  auto product = [&](int M, int N, int K, const float* A, int64_t lda, const float* B, int64_t ldb, bool b_mn,
                     float* C, int64_t ldc, float alpha, bool accumulate) {
    GemmDesc g;
    g.M = M; g.N = N; g.K = K; g.lda = lda; g.ldb = ldb; g.b_mn = b_mn;
    g.a_type = g.b_type = ELEM_F32;
    g.terms[0] = {A, B};
    g.out = OUT_F32; g.C0 = C; g.ldc = ldc; g.alpha = alpha; g.accumulate = accumulate;
    g.gate = c.gate;
    return g;
  };
  const float* W21 = W + (size_t)r1 * ld;
  float* W22 = W + (size_t)r1 * ld + r1;
  float* X22 = X + (size_t)r1 * ld + r1;
  float* X21 = X + (size_t)r1 * ld;
  // L21 = W21 X11^T : C[m][n] = sum_k W21[m][k] X11[n][k]
  LORACT_CUDA_TRY(gemm_f32_small_launch(product(r2, r1, r1, W21, ld, X, ld, false, T1, r1, 1.f, false), c.stream));
  // One launch, two products that both read L21: S = W22 - L21 L21^T (in place) and
  // T2 = L21 X11, T2[m][n] = sum_k L21[m][k] X11[k][n], which the last product below needs.
  {
    const GemmDesc schur = product(r2, r2, r1, T1, r1, T1, r1, false, W22, ld, -1.f, true);
    const GemmDesc l21x11 = product(r2, r1, r1, T1, r1, X, ld, true, T2, r1, 1.f, false);
    LORACT_CUDA_TRY(gemm_f32_small_launch(schur, c.stream, &l21x11));
  }
  LORACT_CUDA_TRY(factor_blocks(c, W22, X22, hi + (size_t)r1 * ld + r1, lo ? lo + (size_t)r1 * ld + r1 : nullptr, r2,
                                Tnext, false));
  // X21 = -X22 T2 : X21[m][n] = -sum_k X22[m][k] T2[k][n], written as fp32 and as the bf16 pair in the same launch
  GemmDesc last = product(r2, r1, r2, X22, ld, T2, r1, true, X21, ld, -1.f, false);
  last.split_hi = hi + (size_t)r1 * ld;
  last.split_lo = lo ? lo + (size_t)r1 * ld : nullptr;
  return gemm_f32_small_launch(last, c.stream);
}

// scratch: W (r x r) + X (r x r) + the temporaries of every level, fp32.
cudaError_t small_block_two_level(const SmallBlockArgs& a, cudaStream_t stream) {
  const int r = a.r;
  float* W = (float*)a.scratch;
  float* X = a.linv_f32 ? a.linv_f32 : W + (size_t)r * r;
  float* T = W + 2 * (size_t)r * r;
  // one launch: W = sum of the partials, and zeros where the blocks above the diagonal are never written below (X is
  // read as a whole by the products of the next level up)
  LORACT_CUDA_TRY(zero3_gated_launch(X, (size_t)r * r * 4, a.linv_hi, (size_t)r * r * 2, a.linv_lo,
                                     a.linv_lo ? (size_t)r * r * 2 : 0, a.gate, stream, (const float*)a.partials,
                                     a.n_partials, a.partial_stride, (int64_t)r * r, W));
  TwoLevelCtx c;
  c.shift_rel = a.shift_rel; c.shift_diag_rel = a.shift_diag_rel; c.gate = a.gate; c.dev_status = a.dev_status; c.ld = r; c.scale_diag = W; c.scale_n = 256;
  c.stream = stream;
  return factor_blocks(c, W, X, a.linv_hi, a.linv_lo, r, T, true);
}

cudaError_t small_block_launch(const SmallBlockArgs& a, cudaStream_t stream) {
  if (small_block_cluster_supported(a)) return small_block_cluster_launch(a, stream);
  if (a.gate_out) return cudaErrorNotSupported;   // only the shared-memory kernel forms the estimate
  if (!a.use_f64 && a.partial_type == ELEM_F32 && a.r > 256 && a.r <= 512 && a.r % 8 == 0 && !a.linv_full &&
      a.linv_hi && a.in_ld == 0 && a.out_ld == 0 && (((uintptr_t)a.partials & 15) == 0) &&
      (a.partial_stride % 4 == 0))
    return small_block_two_level(a, stream);
  if (a.gate) return cudaErrorNotSupported;   // the general kernel is unconditional
  SBParams p;
  p.r = a.r;
  p.partials = a.partials;
  p.partial_is_f64 = a.partial_type == ELEM_F64;
  p.n_partials = a.n_partials;
  p.partial_stride = a.partial_stride;
  p.scratch = a.scratch;
  p.shift_rel = a.shift_rel + a.shift_diag_rel;   // this kernel knows the shift relative to the mean diagonal only
  p.linv_full = a.linv_full;
  p.linv_f32 = a.linv_f32;
  p.linv_hi = a.linv_hi;
  p.linv_lo = a.linv_lo;
  p.dev_status = a.dev_status;
  // Widths above 512 (the comparator with extra test vectors at rank 512) would need a third level of fp32 Schur
  // complements, whose rounding noise reaches the smallest pivots (measured: clamped pivots at 520 columns,
  // non-finite factors at 32768 rows): they take the general kernel in fp64 instead.
  return (a.use_f64 || a.r > 512) ? launch_typed<double>(p, stream) : launch_typed<float>(p, stream);
}

}  // namespace loract

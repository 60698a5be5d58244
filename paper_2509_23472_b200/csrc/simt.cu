// CUDA-core kernels: the generic contraction used by the fp32 path and for shapes the tensor-core
// engine does not take, the fixed-order reduction of split-K partials, and the pre-norm forward.
#include "common.cuh"

namespace loract {

namespace {

template <typename T> __device__ __forceinline__ float load_as_float(const T* p);
template <> __device__ __forceinline__ float load_as_float<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float load_as_float<__nv_bfloat16>(const __nv_bfloat16* p) {
  return __bfloat162float(*p);
}

struct SimtParams {
  int M, N, K;
  int64_t sam, sak;  // element strides of A(m, k)
  int64_t sbk, sbn;  // element strides of B(k, n)
  int n_terms;
  const void* A[4];
  const void* B[4];
  int out;
  void* C0;
  void* C1;
  int64_t ldc;
  int splits;
  int64_t split_stride;
  int accumulate;
  float alpha;
  int halve_at_term;  // the sum so far is multiplied by 1/2 before this term (0: never)
  const uint32_t* gate;  // 32 x 32 tile kernel: optional device word, zero means the launch does nothing
  // 32 x 32 tile kernel: optional bf16 hi / lo copies of the result, same leading dimension as C0
  __nv_bfloat16* split_hi;
  __nv_bfloat16* split_lo;
};

constexpr int kTile = 64;   // output tile 64 x 64, 256 threads, 4 x 4 outputs per thread
constexpr int kTileK = 16;

template <typename TA, typename TB, typename TAcc>
__global__ void __launch_bounds__(256) gemm_simt_kernel(SimtParams p) {
  __shared__ float As[kTileK][kTile + 1];
  __shared__ float Bs[kTileK][kTile + 1];
  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  const int m0 = blockIdx.y * kTile, n0 = blockIdx.x * kTile;
  const int split = blockIdx.z;
  const int k_per = ((p.K + p.splits - 1) / p.splits + kTileK - 1) / kTileK * kTileK;
  const int k_begin = split * k_per;
  const int k_end = min(p.K, k_begin + k_per);
  TAcc acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = (TAcc)0;

  // Each thread loads 4 elements of each operand tile; the faster-varying thread index follows the contiguous
  // dimension of the stored operand.  The next tile is fetched into registers before the current one is
  // multiplied, so the global-memory latency of a tile hides behind the arithmetic of its predecessor.
  for (int term = 0; term < p.n_terms; ++term) {
    const TA* A = (const TA*)p.A[term];
    const TB* B = (const TB*)p.B[term];
    if (term > 0 && term == p.halve_at_term) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] *= (TAcc)0.5;
    }
    float ra[4], rb[4];
    auto fetch = [&](int k0) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = tid + 256 * u;
        int mm, kk;
        if (p.sak == 1) { kk = e % kTileK; mm = e / kTileK; } else { mm = e % kTile; kk = e / kTile; }
        const int m = m0 + mm, k = k0 + kk;
        ra[u] = (m < p.M && k < k_end) ? load_as_float(A + m * p.sam + k * p.sak) : 0.f;
        int nn, kb;
        if (p.sbk == 1) { kb = e % kTileK; nn = e / kTileK; } else { nn = e % kTile; kb = e / kTile; }
        const int n = n0 + nn, k2 = k0 + kb;
        rb[u] = (n < p.N && k2 < k_end) ? load_as_float(B + k2 * p.sbk + n * p.sbn) : 0.f;
      }
    };
    if (k_begin < k_end) fetch(k_begin);
    for (int k0 = k_begin; k0 < k_end; k0 += kTileK) {
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = tid + 256 * u;
        int mm, kk;
        if (p.sak == 1) { kk = e % kTileK; mm = e / kTileK; } else { mm = e % kTile; kk = e / kTile; }
        As[kk][mm] = ra[u];
        int nn, kb;
        if (p.sbk == 1) { kb = e % kTileK; nn = e / kTileK; } else { nn = e % kTile; kb = e / kTile; }
        Bs[kb][nn] = rb[u];
      }
      __syncthreads();
      if (k0 + kTileK < k_end) fetch(k0 + kTileK);
#pragma unroll
      for (int kk = 0; kk < kTileK; ++kk) {
        float a[4], b[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) a[i] = As[kk][ty * 4 + i];
#pragma unroll
        for (int j = 0; j < 4; ++j) b[j] = Bs[kk][tx * 4 + j];
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] += (TAcc)a[i] * (TAcc)b[j];
      }
      __syncthreads();
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + ty * 4 + i;
    if (m >= p.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= p.N) continue;
      const int64_t off = (int64_t)m * p.ldc + n;
      const TAcc v = acc[i][j] * (TAcc)p.alpha;
      if (p.out == OUT_F32) {
        float* c = (float*)p.C0 + (int64_t)split * p.split_stride + off;
        *c = p.accumulate ? (*c + (float)v) : (float)v;
      } else if (p.out == OUT_F64) {
        ((double*)p.C0)[(int64_t)split * p.split_stride + off] = (double)v;
      } else if (p.out == OUT_BF16) {
        ((__nv_bfloat16*)p.C0)[off] = __float2bfloat16((float)v);
      } else {
        const float f = (float)v;
        const __nv_bfloat16 hi = __float2bfloat16(f);
        ((__nv_bfloat16*)p.C0)[off] = hi;
        ((__nv_bfloat16*)p.C1)[off] = __float2bfloat16(f - __bfloat162float(hi));
      }
    }
  }
}

__global__ void reduce_partials_kernel(const float* __restrict__ partials, int n_partials,
                                       int64_t stride, int64_t count, float* __restrict__ out_f32,
                                       __nv_bfloat16* __restrict__ out_bf16, const uint32_t* gate) {
  pdl_wait();
  pdl_launch_dependents();
  if (gate != nullptr && *(const volatile uint32_t*)gate == 0u) return;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
       i += (int64_t)gridDim.x * blockDim.x) {
    float s = 0.f;
    for (int q = 0; q < n_partials; ++q) s += partials[(int64_t)q * stride + i];
    if (out_f32) out_f32[i] = s;
    if (out_bf16) out_bf16[i] = __float2bfloat16(s);
  }
}

// The same sums four elements at a time (16-byte loads, all partials of a quad in flight together): `count4` quads,
// everything 16-byte aligned, stride a multiple of four.  Same order of additions per element as the scalar kernel.
__global__ void __launch_bounds__(256) reduce_partials_vec4_kernel(const float4* __restrict__ partials, int n_partials,
                                                                   int64_t stride4, int64_t count4,
                                                                   float4* __restrict__ out_f32,
                                                                   uint2* __restrict__ out_bf16, const uint32_t* gate) {
  pdl_wait();
  pdl_launch_dependents();
  if (gate != nullptr && *(const volatile uint32_t*)gate == 0u) return;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count4;
       i += (int64_t)gridDim.x * blockDim.x) {
    float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
    int q = 0;
    for (; q + 4 <= n_partials; q += 4) {
      const float4 a = partials[(int64_t)q * stride4 + i], b = partials[(int64_t)(q + 1) * stride4 + i];
      const float4 c = partials[(int64_t)(q + 2) * stride4 + i], d = partials[(int64_t)(q + 3) * stride4 + i];
      s.x = (((s.x + a.x) + b.x) + c.x) + d.x; s.y = (((s.y + a.y) + b.y) + c.y) + d.y;
      s.z = (((s.z + a.z) + b.z) + c.z) + d.z; s.w = (((s.w + a.w) + b.w) + c.w) + d.w;
    }
    for (; q < n_partials; ++q) {
      const float4 a = partials[(int64_t)q * stride4 + i];
      s.x += a.x; s.y += a.y; s.z += a.z; s.w += a.w;
    }
    if (out_f32) out_f32[i] = s;
    if (out_bf16) {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(s.x, s.y), hi = __floats2bfloat162_rn(s.z, s.w);
      out_bf16[i] = make_uint2(*reinterpret_cast<const uint32_t*>(&lo), *reinterpret_cast<const uint32_t*>(&hi));
    }
  }
}

// out = S + S^T with S = sum_s partials[s] (fixed order), for r x r matrices: the tall Gram products are formed as
// D = Yh^T Yh / 2 + Yh^T Yl (two terms), and D + D^T = Yh^T Yh + Yh^T Yl + Yl^T Yh is the three-term Gram matrix,
// exactly symmetric.  One CTA per pair of 16 x 16 tiles (I, J), (J, I), I >= J: both tiles are summed with
// coalesced row reads and meet through shared memory.
constexpr int kSymTile = 16;
// `out` may be the first partial (no __restrict__: see the caller).  1024 threads: two tiles x two halves of the
// partials x 256 elements; a thread adds its partials eight at a time into eight running sums (eight independent
// loads in flight); the sums are combined in a fixed order.
__global__ void __launch_bounds__(1024) reduce_sym_kernel(const float* partials, int n_partials, int64_t stride, int r,
                                                          float* out, const uint32_t* gate) {
  __shared__ float t[2][2][kSymTile][kSymTile + 1];   // [tile][half of the partials][row][column]
  // tile pair from the linear block index: I = largest with I (I + 1) / 2 <= b
  const int b = blockIdx.x;
  int I = 0;
  while ((I + 1) * (I + 2) / 2 <= b) ++I;
  const int J = b - I * (I + 1) / 2;
  const int qh = threadIdx.x >> 9, tile = (threadIdx.x >> 8) & 1;
  const int a = (threadIdx.x >> 4) & 15, c = threadIdx.x & 15;
  // element (a, c) of tile (I, J) (tile 0) or of tile (J, I) (tile 1)
  const int row = (tile ? J : I) * kSymTile + a, col = (tile ? I : J) * kSymTile + c;
  pdl_wait();
  pdl_launch_dependents();
  if (gate != nullptr && *(const volatile uint32_t*)gate == 0u) return;   // the whole grid: this step is not needed
  float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  if (row < r && col < r && !(tile == 1 && I == J)) {
    const float* src = partials + (int64_t)row * r + col;
    const int q_end = qh ? n_partials : n_partials / 2;
    int q = qh ? n_partials / 2 : 0;
    for (; q + 8 <= q_end; q += 8) {
#pragma unroll
      for (int u = 0; u < 8; ++u) acc[u] += src[(int64_t)(q + u) * stride];
    }
    for (int u = 0; q + u < q_end; ++u) acc[u] += src[(int64_t)(q + u) * stride];
  }
  t[tile][qh][a][c] = ((acc[0] + acc[1]) + (acc[2] + acc[3])) + ((acc[4] + acc[5]) + (acc[6] + acc[7]));
  __syncthreads();
  if (qh == 0 && row < r && col < r && !(tile == 1 && I == J)) {
    const int other = (I == J) ? 0 : 1 - tile;
    out[(int64_t)row * r + col] = (t[tile][0][a][c] + t[tile][1][a][c]) + (t[other][0][c][a] + t[other][1][c][a]);
  }
}

// out = sum_s partials[s] (fixed order) written as three bf16 arrays hi + mid + lo (24 mantissa bits), so
// that a tensor-core product with it is as accurate as an fp32 one.  Rows of `cols` elements; the
// partials and the outputs may have different leading dimensions.
__global__ void reduce_split3_kernel(const float* __restrict__ partials, int n_partials, int64_t stride,
                                     int rows, int cols, int64_t ld_in, int64_t ld_out,
                                     __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ mid,
                                     __nv_bfloat16* __restrict__ lo) {
  const int64_t count = (int64_t)rows * cols;
  pdl_wait();
  pdl_launch_dependents();
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < count;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / cols, col = i - row * cols;
    float s = 0.f;
    for (int q = 0; q < n_partials; ++q) s += partials[(int64_t)q * stride + row * ld_in + col];
    const __nv_bfloat16 h = __float2bfloat16(s);
    const float r1 = s - __bfloat162float(h);
    const __nv_bfloat16 m = __float2bfloat16(r1);
    const float r2 = r1 - __bfloat162float(m);
    const int64_t o = row * ld_out + col;
    hi[o] = h; mid[o] = m; lo[o] = __float2bfloat16(r2);
  }
}

// fp32 product for the r x r blocks of the two-level small-block scheme: C = alpha * A B (+ C), all of a few
// hundred rows and columns.  32 x 32 output tiles, four groups of 64 threads per tile, each group on a quarter of
// the contraction (4 x 4 outputs per thread, operands read from shared memory along the contraction index with
// 16-byte loads; the four partial tiles are added in group order), so that a 256 x 256 product spreads over
// 64 SMs and no thread walks more than a quarter of K; the K loop is double-buffered through registers.  One launch carries up to two independent products
// (grid.z picks one): the two-level scheme has a pair of them at one point of its chain.
constexpr int kT32 = 32, kT32Ld = 36;

constexpr int kT32Groups = 4;   // thread groups of 64 that share one output tile, each on a quarter of the contraction
__global__ void __launch_bounds__(64 * kT32Groups) gemm_f32_tile32_kernel(SimtParams p0, SimtParams p1) {
  // per group: As [m][k] and Bs [n][k]; after the K loop the same memory carries the partial tiles of groups 1..3
  __shared__ __align__(16) float tiles[kT32Groups][2][kT32 * kT32Ld];
  const SimtParams& p = blockIdx.z ? p1 : p0;
  const int grp = threadIdx.x >> 6, tid = threadIdx.x & 63;
  float* As = tiles[grp][0];
  float* Bs = tiles[grp][1];
  const int m0 = blockIdx.y * kT32, n0 = blockIdx.x * kT32;
  pdl_wait();
  pdl_launch_dependents();
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) return;
  if (m0 >= p.M || n0 >= p.N) return;
  const int tm = tid >> 3, tn = tid & 7;               // outputs (4 tm + i, tn + 8 j)
  const float* A = (const float*)p.A[0];
  const float* B = (const float*)p.B[0];
  // this group's share of the contraction: whole chunks of 32, the same number of chunks in every group
  const int chunks = ((p.K + kT32 - 1) / kT32 + kT32Groups - 1) / kT32Groups;
  const int k_begin = grp * chunks * kT32;
  const int k_end = min(p.K, k_begin + chunks * kT32);
  float acc[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
  // each thread stages 16 elements of either tile per K chunk; the faster-varying index follows memory
  float ra[16], rb[16];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int e = tid + 64 * u;
      int mm, kk;
      if (p.sak == 1) { kk = e & 31; mm = e >> 5; } else { mm = e & 31; kk = e >> 5; }
      const int m = m0 + mm, k = k0 + kk;
      ra[u] = (m < p.M && k < k_end) ? A[m * p.sam + k * p.sak] : 0.f;
      int nn, kb;
      if (p.sbk == 1) { kb = e & 31; nn = e >> 5; } else { nn = e & 31; kb = e >> 5; }
      const int n = n0 + nn, k2 = k0 + kb;
      rb[u] = (n < p.N && k2 < k_end) ? B[k2 * p.sbk + n * p.sbn] : 0.f;
    }
  };
  auto stash = [&]() {
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const int e = tid + 64 * u;
      int mm, kk;
      if (p.sak == 1) { kk = e & 31; mm = e >> 5; } else { mm = e & 31; kk = e >> 5; }
      As[mm * kT32Ld + kk] = ra[u];
      int nn, kb;
      if (p.sbk == 1) { kb = e & 31; nn = e >> 5; } else { nn = e & 31; kb = e >> 5; }
      Bs[nn * kT32Ld + kb] = rb[u];
    }
  };
  auto group_barrier = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(grp + 1) : "memory"); };
  fetch(k_begin);
  for (int c = 0; c < chunks; ++c) {
    const int k0 = k_begin + c * kT32;
    group_barrier();
    stash();
    group_barrier();
    if (c + 1 < chunks) fetch(k0 + kT32);
#pragma unroll
    for (int q4 = 0; q4 < kT32 / 4; ++q4) {
      float4 a[4], b[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) a[i] = *reinterpret_cast<const float4*>(As + (4 * tm + i) * kT32Ld + 4 * q4);
#pragma unroll
      for (int j = 0; j < 4; ++j) b[j] = *reinterpret_cast<const float4*>(Bs + (tn + 8 * j) * kT32Ld + 4 * q4);
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          acc[i][j] = fmaf(a[i].x, b[j].x, acc[i][j]);
          acc[i][j] = fmaf(a[i].y, b[j].y, acc[i][j]);
          acc[i][j] = fmaf(a[i].z, b[j].z, acc[i][j]);
          acc[i][j] = fmaf(a[i].w, b[j].w, acc[i][j]);
        }
    }
  }
  // the quarters of the contraction meet in shared memory and are added in group order
  group_barrier();   // this group has finished reading its tiles
  if (grp > 0) {
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < 4; ++j) As[(4 * tm + i) * kT32Ld + tn + 8 * j] = acc[i][j];
  }
  __syncthreads();
  if (grp > 0) return;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int m = m0 + 4 * tm + i;
    if (m >= p.M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tn + 8 * j;
      if (n >= p.N) continue;
      float sum = acc[i][j];
#pragma unroll
      for (int g2 = 1; g2 < kT32Groups; ++g2) sum += tiles[g2][0][(4 * tm + i) * kT32Ld + tn + 8 * j];
      float* c = (float*)p.C0 + (int64_t)m * p.ldc + n;
      const float v0 = sum * p.alpha;
      const float v = p.accumulate ? (*c + v0) : v0;
      *c = v;
      if (p.split_hi) {
        const __nv_bfloat16 h = __float2bfloat16(v);
        p.split_hi[(int64_t)m * p.ldc + n] = h;
        if (p.split_lo) p.split_lo[(int64_t)m * p.ldc + n] = __float2bfloat16(v - __bfloat162float(h));
      }
    }
  }
}

// hi/lo split of a block of an fp32 matrix, in place of the same block of two bf16 matrices.
__global__ void split_block_kernel(const float* __restrict__ src, int rows, int cols, int64_t ld,
                                   __nv_bfloat16* __restrict__ hi, __nv_bfloat16* __restrict__ lo,
                                   const uint32_t* gate) {
  if (gate != nullptr && *(const volatile uint32_t*)gate == 0u) return;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < (int64_t)rows * cols;
       i += (int64_t)gridDim.x * blockDim.x) {
    const int64_t row = i / cols, col = i - row * cols;
    const float v = src[row * ld + col];
    const __nv_bfloat16 h = __float2bfloat16(v);
    hi[row * ld + col] = h;
    if (lo) lo[row * ld + col] = __float2bfloat16(v - __bfloat162float(h));
  }
}

// One warp per row: inner = (1 / d) sum_k U[i][k] P[i][k];  row_a = rstd, row_b = rstd * inner.
__global__ void __launch_bounds__(256) rms_backward_rows_kernel(const __nv_bfloat16* __restrict__ U,
                                                                const float* __restrict__ P,
                                                                const float* __restrict__ rstd, int64_t n, int r,
                                                                float inv_d, float* __restrict__ row_a,
                                                                float* __restrict__ row_b) {
  pdl_wait();
  pdl_launch_dependents();
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= n) return;
  float s = 0.f;
  for (int k = lane; k < r; k += 32) s += __bfloat162float(U[row * r + k]) * P[row * r + k];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) {
    const float rs = rstd[row];
    row_a[row] = rs;
    row_b[row] = rs * s * inv_d;
  }
}

// One warp per row.  RMS: rstd = 1/sqrt(mean x^2 + eps).  LayerNorm: mean first, then the centred
// second moment (two passes over the row, which stays in L1/L2), A = (x - mean) rstd gamma + beta.
template <typename T>
__global__ void __launch_bounds__(256) norm_forward_kernel(const T* __restrict__ X, int64_t n, int64_t d,
                                                           int64_t ldx, const T* __restrict__ gamma,
                                                           const T* __restrict__ beta, float eps, int kind,
                                                           T* __restrict__ A, int64_t lda,
                                                           float* __restrict__ rstd_out,
                                                           float* __restrict__ mean_out) {
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= n) return;
  const T* x = X + row * ldx;
  float mean = 0.f;
  if (kind == LORACT_NORM_LAYER) {
    float s = 0.f;
    for (int64_t j = lane; j < d; j += 32) s += load_as_float(x + j);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    mean = s / (float)d;
  }
  float ss = 0.f;
  for (int64_t j = lane; j < d; j += 32) {
    const float v = load_as_float(x + j) - mean;
    ss += v * v;
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float rstd = rsqrtf(ss / (float)d + eps);
  if (lane == 0) {
    rstd_out[row] = rstd;
    if (mean_out) mean_out[row] = mean;
  }
  T* a = A + row * lda;
  for (int64_t j = lane; j < d; j += 32) {
    float v = (load_as_float(x + j) - mean) * rstd * load_as_float(gamma + j);
    if (beta) v += load_as_float(beta + j);
    if constexpr (sizeof(T) == 2) a[j] = __float2bfloat16(v); else a[j] = v;
  }
}

// The same unit with 16-byte accesses, one warp per row.  A lane takes the chunks lane, lane + 32, ... of the
// row (8 bf16 or 4 fp32 values each), so every load and store instruction of a warp covers 512 contiguous
// bytes.  Rows of up to kKeep chunks per lane (d <= 4096 in bf16, 2048 in fp32) stay in registers, packed as
// loaded: X is read from memory exactly once and the statistics (mean, then the centred second moment, as
// in the kernel above) are taken from the registers.  Longer rows are read again for each pass.
constexpr int kNormKeep = 16;

template <typename T>
struct NormChunk;
template <>
struct NormChunk<__nv_bfloat16> {
  static constexpr int kVals = 8;
  static __device__ __forceinline__ void unpack(const uint4& c, float (&v)[8]) {
    const uint32_t w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      v[2 * h] = __uint_as_float(w[h] << 16);
      v[2 * h + 1] = __uint_as_float(w[h] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ uint4 pack(const float (&v)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int h = 0; h < 4; ++h) {
      const __nv_bfloat162 t = __floats2bfloat162_rn(v[2 * h], v[2 * h + 1]);
      w[h] = *reinterpret_cast<const uint32_t*>(&t);
    }
    return make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <>
struct NormChunk<float> {
  static constexpr int kVals = 4;
  static __device__ __forceinline__ void unpack(const uint4& c, float (&v)[4]) {
    v[0] = __uint_as_float(c.x); v[1] = __uint_as_float(c.y); v[2] = __uint_as_float(c.z); v[3] = __uint_as_float(c.w);
  }
  static __device__ __forceinline__ uint4 pack(const float (&v)[4]) {
    return make_uint4(__float_as_uint(v[0]), __float_as_uint(v[1]), __float_as_uint(v[2]), __float_as_uint(v[3]));
  }
};

template <typename T, bool kInRegs>
__global__ void __launch_bounds__(256) norm_forward_vec_kernel(const T* __restrict__ X, int64_t n, int64_t d,
                                                               int64_t ldx, const T* __restrict__ gamma,
                                                               const T* __restrict__ beta, float eps, int kind,
                                                               T* __restrict__ A, int64_t lda,
                                                               float* __restrict__ rstd_out,
                                                               float* __restrict__ mean_out) {
  using C = NormChunk<T>;
  constexpr int kV = C::kVals;
  const int lane = threadIdx.x & 31;
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= n) return;
  const int n_chunks = (int)(d / kV);
  const uint4* x = reinterpret_cast<const uint4*>(X + row * ldx);
  const uint4* gm = reinterpret_cast<const uint4*>(gamma);
  const uint4* bt = reinterpret_cast<const uint4*>(beta);
  uint4* a = reinterpret_cast<uint4*>(A + row * lda);
  uint4 keep[kInRegs ? kNormKeep : 1];
  if (kInRegs) {
#pragma unroll
    for (int i = 0; i < kNormKeep; ++i) {
      const int c = lane + 32 * i;
      keep[i] = c < n_chunks ? x[c] : make_uint4(0u, 0u, 0u, 0u);
    }
  }
  auto chunk = [&](int i, int c) -> uint4 { return kInRegs ? keep[i] : x[c]; };
  const int per_lane = kInRegs ? kNormKeep : (n_chunks + 31) / 32;
  float mean = 0.f;
  if (kind == LORACT_NORM_LAYER) {
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < per_lane; ++i) {
      const int c = lane + 32 * i;
      if (c >= n_chunks) break;
      float v[kV];
      C::unpack(chunk(i, c), v);
#pragma unroll
      for (int q = 0; q < kV; ++q) s += v[q];
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    mean = s / (float)d;
  }
  float ss = 0.f;
#pragma unroll
  for (int i = 0; i < per_lane; ++i) {
    const int c = lane + 32 * i;
    if (c >= n_chunks) break;
    float v[kV];
    C::unpack(chunk(i, c), v);
#pragma unroll
    for (int q = 0; q < kV; ++q) { const float t = v[q] - mean; ss += t * t; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
  const float rstd = rsqrtf(ss / (float)d + eps);
  if (lane == 0) {
    rstd_out[row] = rstd;
    if (mean_out) mean_out[row] = mean;
  }
#pragma unroll
  for (int i = 0; i < per_lane; ++i) {
    const int c = lane + 32 * i;
    if (c >= n_chunks) break;
    float v[kV], g[kV], b[kV];
    C::unpack(chunk(i, c), v);
    C::unpack(__ldg(gm + c), g);
    if (beta) C::unpack(__ldg(bt + c), b);
#pragma unroll
    for (int q = 0; q < kV; ++q) {
      v[q] = (v[q] - mean) * rstd * g[q];
      if (beta) v[q] += b[q];
    }
    a[c] = C::pack(v);
  }
}

template <typename TA, typename TB>
cudaError_t launch_simt_typed(const SimtParams& p, bool acc64, cudaStream_t stream) {
  dim3 grid((p.N + kTile - 1) / kTile, (p.M + kTile - 1) / kTile, p.splits);
  if (acc64) gemm_simt_kernel<TA, TB, double><<<grid, 256, 0, stream>>>(p);
  else gemm_simt_kernel<TA, TB, float><<<grid, 256, 0, stream>>>(p);
  count_launch(__func__, stream);
  return cudaGetLastError();
}

// Decision after the first orthonormalisation round (see round_gate_launch in common.cuh).  One cluster of
// kGateCtas CTAs of 1024 threads; CTA c takes the rows c, c + kGateCtas, ...; a thread takes 8 consecutive elements of
// L^-1 (one 16-byte load) at a time.  Every CTA stores its sum into the shared memory of CTA 0, which adds them in
// rank order after the cluster barrier: a fixed summation order, no state in global memory.
constexpr int kGateCtas = 8;
__global__ void __launch_bounds__(1024) round_gate_kernel(const float* __restrict__ W,
                                                          const __nv_bfloat16* __restrict__ linv_hi, int r,
                                                          float threshold, const uint32_t* dev_status,
                                                          uint32_t* gate_words) {
  __shared__ float s_diag[640];
  __shared__ float s_red[32];
  __shared__ float s_parts[kGateCtas];
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_wait();
  pdl_launch_dependents();
  for (int j = tid; j < r; j += 1024) s_diag[j] = W[(int64_t)j * r + j];
  __syncthreads();
  float acc = 0.f;
  const int groups_per_row = r / 8;       // r is a multiple of 8, so a group of 8 stays inside one row
  // a warp per row: 32 lanes cover 256 columns per step
  for (int row = (int)rank + kGateCtas * warp; row < r; row += kGateCtas * 32) {
    for (int gidx = lane; gidx < groups_per_row && gidx * 8 <= row; gidx += 32) {   // groups that start at or below the diagonal
      const int col = gidx * 8;
      const uint4 v = __ldg(reinterpret_cast<const uint4*>(linv_hi + (int64_t)row * r + col));
      const uint32_t w4[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const float lo = __uint_as_float(w4[q] << 16), hi = __uint_as_float(w4[q] & 0xffff0000u);
        acc += lo * lo * s_diag[col + 2 * q] + hi * hi * s_diag[col + 2 * q + 1];
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) s_red[warp] = acc;
  __syncthreads();
  if (tid == 0) {
    float part = 0.f;
    for (int q = 0; q < 32; ++q) part += s_red[q];
    uint32_t local = (uint32_t)__cvta_generic_to_shared(&s_parts[rank]), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(0));
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(remote), "f"(part) : "memory");
  }
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (rank == 0 && tid == 0) {
    float est = 0.f;
    for (int q = 0; q < kGateCtas; ++q) est += s_parts[q];
    const uint32_t st = dev_status ? *(const volatile uint32_t*)dev_status : 0u;
    const bool again = !(est <= threshold) || st != 0u;   // a NaN estimate compares false: second round
    gate_words[0] = again ? 1u : 0u;
    gate_words[1] = __float_as_uint(est);
    gate_words[2] = again ? 2u : 1u;
  }
}

// Zero fill of up to three 16-byte aligned ranges (counts in 16-byte units) and, in the same launch, an optional
// fixed-order sum of partial matrices (dst[i] = sum_q src[q * stride + i], i < count; count 0: none).  Skipped when
// *gate == 0.
__global__ void zero3_gated_kernel(uint4* a, int64_t na, uint4* b, int64_t nb, uint4* c, int64_t nc,
                                   const float* __restrict__ src, int n_src, int64_t src_stride, int64_t count,
                                   float* __restrict__ dst, const uint32_t* gate) {
  pdl_wait();
  pdl_launch_dependents();
  if (gate != nullptr && *(const volatile uint32_t*)gate == 0u) return;
  const uint4 z = make_uint4(0u, 0u, 0u, 0u);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x, t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  for (int64_t i = t0; i < count; i += stride) {
    float sum = 0.f;
    for (int q = 0; q < n_src; ++q) sum += src[(int64_t)q * src_stride + i];
    dst[i] = sum;
  }
  for (int64_t i = t0; i < na; i += stride) a[i] = z;
  for (int64_t i = t0; i < nb; i += stride) b[i] = z;
  for (int64_t i = t0; i < nc; i += stride) c[i] = z;
}

__global__ void copy_bf16_gated_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst, int64_t n16,
                                       const uint32_t* gate) {
  pdl_wait();
  pdl_launch_dependents();
  if (*(const volatile uint32_t*)gate == 0u) return;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (int64_t)gridDim.x * blockDim.x)
    dst[i] = src[i];
}

}  // namespace

cudaError_t gemm_simt_launch(const GemmDesc& g, cudaStream_t stream) {
  SimtParams p;
  p.M = g.M; p.N = g.N; p.K = g.K;
  if (g.a_mn) { p.sam = 1; p.sak = g.lda; } else { p.sam = g.lda; p.sak = 1; }
  if (g.b_mn) { p.sbn = 1; p.sbk = g.ldb; } else { p.sbn = g.ldb; p.sbk = 1; }
  p.n_terms = g.n_terms;
  for (int t = 0; t < 4; ++t) { p.A[t] = g.terms[t].A; p.B[t] = g.terms[t].B; }
  p.out = g.out; p.C0 = g.C0; p.C1 = g.C1; p.ldc = g.ldc;
  p.splits = g.splits < 1 ? 1 : g.splits;
  p.split_stride = g.split_stride;
  p.accumulate = g.accumulate ? 1 : 0;
  p.alpha = g.alpha;
  p.halve_at_term = g.halve_at_term > 0 ? g.halve_at_term : 0;
  if (p.splits > 1 && !(g.out == OUT_F32 || g.out == OUT_F64)) return cudaErrorInvalidValue;
  const bool a16 = g.a_type == ELEM_BF16, b16 = g.b_type == ELEM_BF16;
  if (a16 && b16) return launch_simt_typed<__nv_bfloat16, __nv_bfloat16>(p, g.acc64, stream);
  if (a16 && !b16) return launch_simt_typed<__nv_bfloat16, float>(p, g.acc64, stream);
  if (!a16 && b16) return launch_simt_typed<float, __nv_bfloat16>(p, g.acc64, stream);
  return launch_simt_typed<float, float>(p, g.acc64, stream);
}

cudaError_t reduce_partials_launch(const float* partials, int n_partials, int64_t stride,
                                   int64_t count, float* out_f32, __nv_bfloat16* out_bf16,
                                   cudaStream_t stream, const uint32_t* gate) {
  // four elements per thread only where that still leaves a few CTAs per SM (a small matrix is summed faster by
  // more threads with one element each)
  const bool vec = count >= (1 << 18) && count % 4 == 0 && stride % 4 == 0 &&
                   (((uintptr_t)partials | (uintptr_t)out_f32) & 15) == 0 && ((uintptr_t)out_bf16 & 7) == 0;
  if (vec) {
    const int64_t count4 = count / 4;
    int grid = (int)((count4 + 255) / 256);
    if (grid > 148 * 8) grid = 148 * 8;
    if (grid < 1) grid = 1;
    LORACT_CUDA_TRY(launch_pdl(reduce_partials_vec4_kernel, dim3(grid), dim3(256), 0, stream, (const float4*)partials,
                               n_partials, stride / 4, count4, (float4*)out_f32, (uint2*)out_bf16, gate));
    count_launch(__func__, stream);
    return cudaGetLastError();
  }
  int grid = (int)((count + 255) / 256);
  if (grid > 148 * 16) grid = 148 * 16;
  if (grid < 1) grid = 1;
  LORACT_CUDA_TRY(launch_pdl(reduce_partials_kernel, dim3(grid), dim3(256), 0, stream, partials, n_partials, stride,
                             count, out_f32, out_bf16, gate));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t reduce_sym_launch(const float* partials, int n_partials, int64_t stride, int r, float* out,
                              cudaStream_t stream, const uint32_t* gate) {
  const int nt = (r + kSymTile - 1) / kSymTile;
  LORACT_CUDA_TRY(launch_pdl(reduce_sym_kernel, dim3(nt * (nt + 1) / 2), dim3(1024), 0, stream, partials, n_partials,
                             stride, r, out, gate));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t round_gate_launch(const float* W, const __nv_bfloat16* linv_hi, int r, float threshold,
                              const uint32_t* dev_status, uint32_t* gate_words, cudaStream_t stream) {
  if (r < 8 || r > 640 || r % 8 || ((uintptr_t)linv_hi & 15)) return cudaErrorInvalidValue;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kGateCtas, 1, 1);
  cfg.blockDim = dim3(1024, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kGateCtas;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  LORACT_CUDA_TRY(cudaLaunchKernelEx(&cfg, round_gate_kernel, W, linv_hi, r, threshold, dev_status, gate_words));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t zero3_gated_launch(void* a, size_t a_bytes, void* b, size_t b_bytes, void* c, size_t c_bytes,
                               const uint32_t* gate, cudaStream_t stream, const float* sum_src, int n_src,
                               int64_t src_stride, int64_t count, float* sum_dst) {
  if (((uintptr_t)a | (uintptr_t)b | (uintptr_t)c | a_bytes | b_bytes | c_bytes) & 15) return cudaErrorInvalidValue;
  LORACT_CUDA_TRY(launch_pdl(zero3_gated_kernel, dim3(148), dim3(512), 0, stream, (uint4*)a, (int64_t)(a_bytes / 16),
                             (uint4*)b, (int64_t)(b_bytes / 16), (uint4*)c, (int64_t)(c_bytes / 16), sum_src, n_src,
                             src_stride, sum_src ? count : (int64_t)0, sum_dst, gate));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t copy_bf16_gated_launch(const __nv_bfloat16* src, __nv_bfloat16* dst, int64_t count, const uint32_t* gate,
                                   cudaStream_t stream) {
  if (count % 8 || ((uintptr_t)src & 15) || ((uintptr_t)dst & 15) || !gate) return cudaErrorInvalidValue;
  const int64_t n16 = count / 8;
  int grid = (int)((n16 + 255) / 256);
  if (grid > 148 * 8) grid = 148 * 8;
  if (grid < 1) grid = 1;
  LORACT_CUDA_TRY(launch_pdl(copy_bf16_gated_kernel, dim3(grid), dim3(256), 0, stream, (const uint4*)src, (uint4*)dst,
                             n16, gate));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t reduce_split3_launch(const float* partials, int n_partials, int64_t stride, int rows, int cols,
                                 int64_t ld_in, int64_t ld_out, __nv_bfloat16* hi, __nv_bfloat16* mid,
                                 __nv_bfloat16* lo, cudaStream_t stream) {
  int grid = (int)(((int64_t)rows * cols + 255) / 256);
  if (grid > 148 * 8) grid = 148 * 8;
  if (grid < 1) grid = 1;
  LORACT_CUDA_TRY(launch_pdl(reduce_split3_kernel, dim3(grid), dim3(256), 0, stream, partials, n_partials, stride, rows,
                             cols, ld_in, ld_out, hi, mid, lo));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t gemm_f32_small_launch(const GemmDesc& g, cudaStream_t stream, const GemmDesc* second) {
  auto fill = [](const GemmDesc& g, SimtParams& p) {
    // (the gate of the first product holds for the whole launch)
    if (g.a_type != ELEM_F32 || g.b_type != ELEM_F32 || g.out != OUT_F32 || g.n_terms != 1 || g.splits > 1)
      return false;
    p = SimtParams{};
    p.M = g.M; p.N = g.N; p.K = g.K;
    if (g.a_mn) { p.sam = 1; p.sak = g.lda; } else { p.sam = g.lda; p.sak = 1; }
    if (g.b_mn) { p.sbn = 1; p.sbk = g.ldb; } else { p.sbn = g.ldb; p.sbk = 1; }
    p.n_terms = 1;
    p.A[0] = g.terms[0].A; p.B[0] = g.terms[0].B;
    p.out = g.out; p.C0 = g.C0; p.ldc = g.ldc; p.splits = 1;
    p.accumulate = g.accumulate ? 1 : 0;
    p.alpha = g.alpha;
    p.gate = nullptr;
    p.split_hi = (__nv_bfloat16*)g.split_hi;
    p.split_lo = (__nv_bfloat16*)g.split_lo;
    return true;
  };
  SimtParams p0, p1;
  if (!fill(g, p0) || (second && !fill(*second, p1))) return cudaErrorNotSupported;
  if (!second) p1 = p0;
  p0.gate = p1.gate = g.gate;
  const int M = second ? std::max(g.M, second->M) : g.M, N = second ? std::max(g.N, second->N) : g.N;
  dim3 grid((N + kT32 - 1) / kT32, (M + kT32 - 1) / kT32, second ? 2 : 1);
  LORACT_CUDA_TRY(launch_pdl(gemm_f32_tile32_kernel, grid, dim3(64 * kT32Groups), 0, stream, p0, p1));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t split_block_launch(const float* src, int rows, int cols, int64_t ld, __nv_bfloat16* hi,
                               __nv_bfloat16* lo, cudaStream_t stream, const uint32_t* gate) {
  int grid = (int)(((int64_t)rows * cols + 255) / 256);
  if (grid > 148 * 4) grid = 148 * 4;
  split_block_kernel<<<grid, 256, 0, stream>>>(src, rows, cols, ld, hi, lo, gate);
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t rms_backward_rows_launch(const __nv_bfloat16* U, const float* P, const float* rstd, int64_t n, int r,
                                     int64_t d, float* row_a, float* row_b, cudaStream_t stream) {
  const int warps = 8;
  const int grid = (int)((n + warps - 1) / warps);
  LORACT_CUDA_TRY(launch_pdl(rms_backward_rows_kernel, dim3(grid), dim3(warps * 32), 0, stream, U, P, rstd, n, r,
                             1.0f / (float)d, row_a, row_b));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t norm_forward_launch(const void* X, int64_t n, int64_t d, int64_t ldx, int elem_type,
                                const void* gamma, const void* beta, float eps, int kind, void* A,
                                int64_t lda, float* rstd, float* mean, cudaStream_t stream) {
  const int warps = 8;
  const int grid = (int)((n + warps - 1) / warps);
  const int vals = elem_type == ELEM_BF16 ? 8 : 4;
  // 16-byte accesses need every row of X and A, and gamma and beta, on a 16-byte boundary
  const bool vec = d % vals == 0 && ldx % vals == 0 && lda % vals == 0 && (((uintptr_t)X | (uintptr_t)A |
                   (uintptr_t)gamma | (uintptr_t)beta) & 15) == 0;
  const bool in_regs = d <= (int64_t)vals * 32 * kNormKeep;
  if (elem_type == ELEM_BF16) {
    typedef __nv_bfloat16 T;
    if (vec && in_regs)
      norm_forward_vec_kernel<T, true><<<grid, warps * 32, 0, stream>>>((const T*)X, n, d, ldx, (const T*)gamma,
                                                                       (const T*)beta, eps, kind, (T*)A, lda, rstd, mean);
    else if (vec)
      norm_forward_vec_kernel<T, false><<<grid, warps * 32, 0, stream>>>((const T*)X, n, d, ldx, (const T*)gamma,
                                                                        (const T*)beta, eps, kind, (T*)A, lda, rstd, mean);
    else
      norm_forward_kernel<T><<<grid, warps * 32, 0, stream>>>((const T*)X, n, d, ldx, (const T*)gamma, (const T*)beta,
                                                              eps, kind, (T*)A, lda, rstd, mean);
  } else {
    typedef float T;
    if (vec && in_regs)
      norm_forward_vec_kernel<T, true><<<grid, warps * 32, 0, stream>>>((const T*)X, n, d, ldx, (const T*)gamma,
                                                                       (const T*)beta, eps, kind, (T*)A, lda, rstd, mean);
    else if (vec)
      norm_forward_vec_kernel<T, false><<<grid, warps * 32, 0, stream>>>((const T*)X, n, d, ldx, (const T*)gamma,
                                                                        (const T*)beta, eps, kind, (T*)A, lda, rstd, mean);
    else
      norm_forward_kernel<T><<<grid, warps * 32, 0, stream>>>((const T*)X, n, d, ldx, (const T*)gamma, (const T*)beta,
                                                              eps, kind, (T*)A, lda, rstd, mean);
  }
  count_launch(__func__, stream);
  return cudaGetLastError();
}

}  // namespace loract

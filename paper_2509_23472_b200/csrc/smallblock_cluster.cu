// Small-block factorisation for r <= 256, fp32: Cholesky factor of an r x r Gram matrix and the inverse
// of that factor (the serial part of the orthonormalisation, the QR step of Algorithm 1 done through Gram
// matrices), as one thread-block-cluster kernel whose working set never leaves shared memory.
//
// The matrix is cut into 32 x 32 blocks.  Eight CTAs form a cluster:
//   * CTA 0 is the pivot chain.  For block column k two warps factor the diagonal block in registers
//     (one the columns 0..15, one the columns 16..31) while eight more invert the factor alongside; the
//     CTA then forms L(k+1,k) = A(k+1,k) D_k^{-T} and applies it to the next diagonal block itself, so the
//     chain waits for nothing but the two blocks it needs next.  One more warp only sends.
//   * CTAs 1..7 own all blocks (dealt out column by column).  Half of their warps do the factorisation:
//     for column k each forms its L(i,k), then updates its trailing blocks, A(i,j) -= L(i,k) L(j,k)^T; the
//     two blocks the chain needs next, (k+2,k+1) and (k+2,k+2), are updated first and sent to CTA 0.
//     The other half computes the inverse X = L^{-1} by block columns, right-looking: block row k becomes
//     final at step k, X(k,j) = -D_k^{-1} T(k,j), is written out and added into the sums of the later rows,
//     T(i,j) += L(i,k) X(k,j).  It stands back while the first half is on the chain's critical path.
//   * Every finished block (D_k^{-1}, L(i,k)) is copied into the same slot of every worker's shared memory
//     with bulk distributed-shared-memory copies (cp.async.bulk shared::cta -> shared::cluster) that count
//     bytes on an mbarrier of the receiving CTA, so each worker ends up with a full copy of L without a
//     global-memory round trip, a fence or a remote arrive.  (16-byte st.async stores were tried first:
//     one barrier update per 16 bytes made the sends the bottleneck.)
//   * 32 x 32 block products run on CUDA cores with 4 x 4 (or 2 x 2) outputs per thread; they are bound by
//     shared-memory bandwidth (a 16-byte load costs about four cycles of the pipe), hence the tiling.
// Every wait is bounded (a wall-clock limit for barriers, an iteration limit for flag words); on expiry the
// CTA records LORACT_DEV_WAIT_EXPIRED, stops waiting and runs to its end (results are then invalid but
// every access stays in bounds).
#include <atomic>

#include "common.cuh"

namespace loract {

namespace {

constexpr int kB = 32;                   // block edge
constexpr int kLd = 36;                  // padded row stride of a block slot (floats): rows 16-byte aligned
constexpr int kSlot = kB * kLd;          // floats per slot
constexpr int kSlotTx = kSlot * 4;        // bytes one sent block (padding included) adds to a barrier's transaction count
constexpr int kMaxBlk = 8;               // r <= 256
constexpr int kCl = 8;                   // CTAs per cluster
constexpr int kWorkers = kCl - 1;
constexpr int kCThreads = 512;
constexpr int kGroup = 256;              // threads of a warp group (8 warps, 4 block rows each)
constexpr int kMaxTri = kMaxBlk * (kMaxBlk + 1) / 2;
constexpr int kXSlots = kMaxBlk;         // inverse blocks of the block columns one CTA owns
constexpr uint64_t kClusterWaitNs = 50000000ull;  // 50 ms

struct SCParams {
  int r;
  const float* partials;
  int n_partials;
  int64_t partial_stride;
  float shift_rel;
  float shift_diag_rel;    // each diagonal entry is also multiplied by (1 + shift_diag_rel)
  const uint32_t* gate;    // optional device word: zero means every CTA leaves at once
  // optional: three words that receive the decision on a further orthonormalisation round
  // { est > gate_threshold or est not finite or *dev_status != 0, est as float bits, 1 or 2 },
  // est = sum_ij Linv_ij^2 W_jj (W_jj the diagonal as factored): trace of the inverse of the diagonally scaled matrix
  uint32_t* gate_out;
  float gate_threshold;
  float* linv_f32;
  __nv_bfloat16* linv_hi;
  __nv_bfloat16* linv_lo;
  uint32_t* dev_status;
  int64_t in_ld, out_ld;   // row strides of the partial matrices and of the outputs
  const float* scale_diag; // optional: another matrix whose diagonal sets the scale of shift and floor
  int scale_n;
  int64_t scale_ld;
};

__device__ __forceinline__ int tri(int i, int j) { return i * (i + 1) / 2 + j; }

// Worker (1..7) that owns block (i, j), i >= j: blocks are dealt out in column-major order, so the blocks
// of one column sit on different CTAs.
__device__ __forceinline__ int owner_of(int i, int j, int nblk) {
  const int n = j * nblk - j * (j - 1) / 2 + (i - j);
  return 1 + n % kWorkers;
}

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t map_to_cta(uint32_t local_addr, int rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, float4 v) {
  asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z),
               "f"(v.w)
               : "memory");
}
__device__ __forceinline__ void bar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
}
__device__ __forceinline__ void bar_expect(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bar_arrive_local(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool bar_try(uint64_t* bar) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], 0;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_addr(bar))
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Every barrier of this kernel completes exactly once (phase 0).  Called by ONE thread of a warp group;
// the others block on the named barrier that follows, so that waiting costs no issue slots.  Returns
// false once the CTA has given up.
__device__ __forceinline__ bool bar_wait(uint64_t* bar, volatile int* gave_up, uint64_t limit_ns = kClusterWaitNs) {
  if (bar_try(bar)) return true;
  if (*gave_up) return false;
  uint64_t t0 = 0;
  for (uint32_t spin = 1;; ++spin) {
    if (bar_try(bar)) return true;
    __nanosleep(20);
    if ((spin & 255u) == 0u) {
      if (*gave_up) return false;
      const uint64_t now = timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) { *gave_up = 1; return false; }
    }
  }
}
__device__ __forceinline__ void group_sync(int id) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(kGroup) : "memory");
}
__device__ __forceinline__ void chain_sync() { asm volatile("bar.sync 3, 352;" ::: "memory"); }   // warps 0..10 of CTA 0
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// 32 x 32 block product C += A B^T on (32 / TM) * (32 / TN) threads, thread t of them holding the TM x TN
// outputs C[TM tm + i][tn + NT j], NT = 32 / TN, tm = t / NT, tn = t % NT.  Both operands are read along
// the contraction index with 16-byte loads: TM + TN loads feed 4 TM TN FMAs, which is what keeps the
// shared-memory pipe (the limit of these products) below the FMA pipe.  The eight lanes of a quarter
// warp read one row of A (a broadcast) and eight different rows of B, whose stride of 36 words spreads
// them over all banks.
template <int TM, int TN>
__device__ __forceinline__ void tile_mac(float (&acc)[TM][TN], const float* __restrict__ A,
                                         const float* __restrict__ Bm, int tm, int tn) {
  constexpr int NT = kB / TN;
#pragma unroll
  for (int q4 = 0; q4 < kB / 4; ++q4) {
    float4 a[TM], b[TN];
#pragma unroll
    for (int i = 0; i < TM; ++i) a[i] = *reinterpret_cast<const float4*>(A + (TM * tm + i) * kLd + 4 * q4);
#pragma unroll
    for (int j = 0; j < TN; ++j) b[j] = *reinterpret_cast<const float4*>(Bm + (tn + NT * j) * kLd + 4 * q4);
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
      for (int j = 0; j < TN; ++j) {
        acc[i][j] = fmaf(a[i].x, b[j].x, acc[i][j]);
        acc[i][j] = fmaf(a[i].y, b[j].y, acc[i][j]);
        acc[i][j] = fmaf(a[i].z, b[j].z, acc[i][j]);
        acc[i][j] = fmaf(a[i].w, b[j].w, acc[i][j]);
      }
  }
}
template <int TM, int TN>
__device__ __forceinline__ void tile_zero(float (&acc)[TM][TN]) {
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;
}
// dst[TM tm + i][tn + NT j] = alpha * acc[i][j] + beta * dst[...]
template <int TM, int TN>
__device__ __forceinline__ void tile_store(float* dst, const float (&acc)[TM][TN], int tm, int tn, float alpha,
                                           bool add) {
  constexpr int NT = kB / TN;
#pragma unroll
  for (int i = 0; i < TM; ++i)
#pragma unroll
    for (int j = 0; j < TN; ++j) {
      float* d = dst + (TM * tm + i) * kLd + tn + NT * j;
      *d = add ? fmaf(alpha, acc[i][j], *d) : alpha * acc[i][j];
    }
}

// Bulk copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) from this CTA's shared memory
// into a peer's; on arrival `bytes` is taken off the transaction count of the peer's barrier `bar`.
__device__ __forceinline__ void bulk_to_peer(uint32_t dst_cluster_addr, uint32_t src_local_addr, uint32_t bytes,
                                             uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
      ::"r"(dst_cluster_addr), "r"(src_local_addr), "r"(bytes), "r"(bar_cluster_addr)
      : "memory");
}
__device__ __forceinline__ void fence_async_proxy() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// One warp has just written rows [row0, row0 + n_rows) of the block in `slot_local` (plain stores, every
// lane has executed fence_async_proxy).  Lanes first_dst .. last_dst (except `skip`) each copy those rows
// into the same slot of the CTA with their number, counting the bytes on that CTA's barrier `bar_local`.
__device__ __forceinline__ void send_rows(const float* slot_local, int row0, int n_rows, const uint64_t* bar_local,
                                          int first_dst, int last_dst, int skip, int lane) {
  __syncwarp();
  if (lane >= first_dst && lane <= last_dst && lane != skip) {
    const uint32_t src = smem_addr(slot_local + row0 * kLd);
    bulk_to_peer(map_to_cta(src, lane), src, (uint32_t)(n_rows * kLd * 4),
                 map_to_cta(smem_addr(bar_local), lane));
  }
}

// The 32 x 32 diagonal block is handled by ten warps that run side by side: two factor it (one the
// columns 0..15, one the columns 16..31), eight invert the factor, four columns each.  Straight-line
// code like this runs at the rate instructions can be fetched, so the work per column is spread thin;
// what remains per column is the latency of the pivot (broadcast, reciprocal square root, one FMA).
//
// As soon as column k of L is known it is published twice, both arrays starting out as kUnset so that a
// consumer needs no flag and no fence -- it waits for its word to change:
//   lcol[k][i] = L[i][k] (i > k), 1 / L[k][k] (i = k), 0 (i < k)             for the other factor warp
//   mcol[k][i] = L[i][k] / L[k][k] (i > k), 1 / L[k][k] (i = k), 0 (i < k)   for the inverting warps
constexpr uint32_t kUnset = 0xFFFFFFFFu;   // a NaN pattern arithmetic does not produce
constexpr int kLcolLd = kLd;              // rows of `lcol` are read back as float4
constexpr int kHalf = kB / 2;
constexpr int kInvWarps = 8;
constexpr int kInvCols = kB / kInvWarps;  // columns of the inverse one of those warps holds

// One MUFU instruction (2 ulp); the argument is a clamped, positive, normal pivot.
__device__ __forceinline__ float fast_rsqrt(float x) {
  float y;
  asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float not_unset(float v) { return __float_as_uint(v) == kUnset ? 0.f : v; }

// Bounded wait for one word of lcol / mcol.
__device__ __forceinline__ float wait_word(const float* addr, volatile int* gave_up) {
  const volatile uint32_t* src = reinterpret_cast<const volatile uint32_t*>(addr);
  uint32_t bits = *src;
  for (uint32_t spin = 0; bits == kUnset; ++spin) {
    if (spin > (1u << 20) || *gave_up) { *gave_up = 1; bits = 0u; break; }
    __nanosleep(32);   // a warp that spins would take issue slots from the factoring warp next to it
    bits = *src;
  }
  return __uint_as_float(bits);
}

// One pivot column of the right-looking Cholesky inside a warp that holds the columns [c0, c0 + 16) of
// every row (lane = row) as float2 pairs `a2`: takes the pivot's reciprocal square root `rinv`, forms and
// publishes the column, updates the later columns of this warp with 16-byte broadcast loads and packed
// FMAs, and starts the next pivot early.  K is the column inside the warp's range (compile time).
template <int K>
__device__ __forceinline__ void pivot_column(float2 (&a2)[kHalf / 2], float& diag, float& rinv, bool& bad,
                                             bool& clamped, int c0, float* lcol, float* mcol, float pivot_floor,
                                             int lane) {
  const int k = c0 + K;
  const float ak = (K & 1) ? a2[K >> 1].y : a2[K >> 1].x;
  // a pivot that is not safely positive was replaced by the floor; its column is dropped (entries below
  // such a pivot are rounding noise; dividing them by the tiny pivot would overflow later columns)
  const float lik = (lane > k && !bad) ? ak * rinv : 0.f;   // L[lane][k]
  lcol[k * kLcolLd + lane] = not_unset((lane == k) ? rinv : lik);
  mcol[k * kLcolLd + lane] = not_unset((lane == k) ? rinv : lik * rinv);
  diag = fmaf(-lik, lik, diag);
  if (K + 1 < kHalf) {
    // the next column first, through a shuffle (shorter than the round trip through shared memory), and
    // the next pivot straight away: its square root is in flight while the rest of this column's
    // updates are issued
    const float l1 = __shfl_sync(0xffffffffu, lik, k + 1);
    if ((K + 1) & 1) a2[(K + 1) >> 1].y = fmaf(-lik, l1, a2[(K + 1) >> 1].y);
    else a2[(K + 1) >> 1].x = fmaf(-lik, l1, a2[(K + 1) >> 1].x);
    float an = __shfl_sync(0xffffffffu, diag, k + 1);
    bad = !(an > pivot_floor);
    if (bad) { an = pivot_floor; clamped = true; }
    rinv = fast_rsqrt(an);
    __syncwarp();
    const float2 nl = make_float2(-lik, -lik);
    const float4* col = reinterpret_cast<const float4*>(lcol + k * kLcolLd + c0);
    // columns K + 2 ..: 16-byte broadcast loads of the published column, packed FMAs.  In the quad that
    // holds column K + 1 the entries up to it are masked out (K + 1 is done, earlier ones are not read).
    constexpr int q1 = (K + 2) >> 2;
#pragma unroll
    for (int q = q1; q < kHalf / 4; ++q) {
      float4 l2 = col[q];
      if (4 * q + 0 < K + 2) l2.x = 0.f;
      if (4 * q + 1 < K + 2) l2.y = 0.f;
      if (4 * q + 2 < K + 2) l2.z = 0.f;
      if (4 * q + 3 < K + 2) l2.w = 0.f;
      a2[2 * q] = __ffma2_rn(nl, make_float2(l2.x, l2.y), a2[2 * q]);
      a2[2 * q + 1] = __ffma2_rn(nl, make_float2(l2.z, l2.w), a2[2 * q + 1]);
    }
  }
}

template <int K>
__device__ __forceinline__ void pivot_columns_from(float2 (&a2)[kHalf / 2], float& diag, float& rinv, bool& bad,
                                                   bool& clamped, int c0, float* lcol, float* mcol,
                                                   float pivot_floor, int lane) {
  if constexpr (K < kHalf) {
    pivot_column<K>(a2, diag, rinv, bad, clamped, c0, lcol, mcol, pivot_floor, lane);
    pivot_columns_from<K + 1>(a2, diag, rinv, bad, clamped, c0, lcol, mcol, pivot_floor, lane);
  }
}

// Factor warp `half` (0: columns 0..15, 1: columns 16..31) of the diagonal block in `slot`.  The second
// warp first follows the columns the first one publishes, taking them off its own columns, then carries
// on with the pivots 16..31.  Returns true if a pivot was clamped.
__device__ __forceinline__ bool factor_diag_half(const float* slot, float* lcol, float* mcol, float pivot_floor,
                                                 volatile int* gave_up, int half, int lane) {
  const int c0 = half * kHalf;
  float2 a2[kHalf / 2];   // row `lane`, columns (c0 + 2p, c0 + 2p + 1), below the diagonal only
  float diag = slot[lane * kLd + lane];   // used by the lanes whose diagonal lies in this warp's columns
  if (half == 0) {
#pragma unroll
    for (int pp = 0; pp < kHalf / 2; ++pp)
      a2[pp] = make_float2(2 * pp < lane ? slot[lane * kLd + 2 * pp] : 0.f,
                           2 * pp + 1 < lane ? slot[lane * kLd + 2 * pp + 1] : 0.f);
  } else {
    // The following warp.  Rows 0..15 have nothing below the diagonal in the columns 16..31, so their lanes
    // would idle: instead lane i and lane i - 16 share row i while the columns of the first warp are taken
    // off (lane i its columns 16..23, lane i - 16 the columns 24..31), which halves the instructions per
    // followed column -- this warp ran a thousand cycles behind the one it follows -- and the upper lanes
    // collect the whole row with eight shuffles before their own pivots start.  Two columns are taken per
    // round trip: the updates commute (both use final values of L) and their loads overlap.
    const int row = lane | kHalf;
    const int cb = kHalf + ((lane < kHalf) ? kHalf / 2 : 0);   // first of this lane's eight columns
    float2 f[kHalf / 4];
#pragma unroll
    for (int pp = 0; pp < kHalf / 4; ++pp)
      f[pp] = make_float2(cb + 2 * pp < row ? slot[row * kLd + cb + 2 * pp] : 0.f,
                          cb + 2 * pp + 1 < row ? slot[row * kLd + cb + 2 * pp + 1] : 0.f);
#pragma unroll
    for (int k = 0; k < kHalf; k += 2) {
      const float l0 = wait_word(lcol + k * kLcolLd + row, gave_up);         // L[row][k]
      const float l1 = wait_word(lcol + (k + 1) * kLcolLd + row, gave_up);   // L[row][k + 1]
      __syncwarp();
      const float2 n0 = make_float2(-l0, -l0), n1 = make_float2(-l1, -l1);
      const float4* c0p = reinterpret_cast<const float4*>(lcol + k * kLcolLd + cb);
      const float4* c1p = reinterpret_cast<const float4*>(lcol + (k + 1) * kLcolLd + cb);
      const float4 la0 = c0p[0], la1 = c0p[1], lb0 = c1p[0], lb1 = c1p[1];
      if (lane >= kHalf) diag = fmaf(-l1, l1, fmaf(-l0, l0, diag));
      f[0] = __ffma2_rn(n0, make_float2(la0.x, la0.y), f[0]);
      f[1] = __ffma2_rn(n0, make_float2(la0.z, la0.w), f[1]);
      f[2] = __ffma2_rn(n0, make_float2(la1.x, la1.y), f[2]);
      f[3] = __ffma2_rn(n0, make_float2(la1.z, la1.w), f[3]);
      f[0] = __ffma2_rn(n1, make_float2(lb0.x, lb0.y), f[0]);
      f[1] = __ffma2_rn(n1, make_float2(lb0.z, lb0.w), f[1]);
      f[2] = __ffma2_rn(n1, make_float2(lb1.x, lb1.y), f[2]);
      f[3] = __ffma2_rn(n1, make_float2(lb1.z, lb1.w), f[3]);
    }
#pragma unroll
    for (int pp = 0; pp < kHalf / 4; ++pp) {
      // columns 24..31 of row `lane` come up from lane - 16 (the source lane wraps for the lower lanes,
      // whose registers are cleared right after)
      const float tx = __shfl_sync(0xffffffffu, f[pp].x, (lane + kHalf) & 31);
      const float ty = __shfl_sync(0xffffffffu, f[pp].y, (lane + kHalf) & 31);
      a2[pp] = (lane >= kHalf) ? f[pp] : make_float2(0.f, 0.f);
      a2[kHalf / 4 + pp] = (lane >= kHalf) ? make_float2(tx, ty) : make_float2(0.f, 0.f);
    }
  }
  bool clamped = false;
  float akk = __shfl_sync(0xffffffffu, diag, c0);
  bool bad = !(akk > pivot_floor);
  if (bad) { akk = pivot_floor; clamped = true; }
  float rinv = fast_rsqrt(akk);
  pivot_columns_from<0>(a2, diag, rinv, bad, clamped, c0, lcol, mcol, pivot_floor, lane);
  return clamped;
}

// Inverting warp `part` (lane i holds row i of X = L^{-1}, columns 4 part .. 4 part + 3): takes the scaled
// columns of L as they appear in `mcol` and works right-looking: once column k is known, row k of X is
// final up to its scale 1 / L[k][k], and every later row takes L[i][k] / L[k][k] times the unscaled row k
// (four shuffles from lane k) off -- no serial dot products.  Columns k < 4 part cannot touch this warp's
// columns and are skipped.  Writes its columns of X (lower triangular, zeros above) into `slot`.
__device__ __forceinline__ void invert_diag_part(float* slot, const float* mcol, volatile int* gave_up, int part,
                                                 int lane) {
  const int j0 = part * kInvCols;
  float2 x01 = make_float2(j0 == lane ? 1.f : 0.f, j0 + 1 == lane ? 1.f : 0.f);
  float2 x23 = make_float2(j0 + 2 == lane ? 1.f : 0.f, j0 + 3 == lane ? 1.f : 0.f);
  float my_rinv = 1.f;
  // Four columns per round: the words of all four are fetched together (and waited for only if one is still
  // unset), then the four updates run back to back with nothing in them but the broadcast of row k and two
  // packed FMAs.  One column per round cost about 180 cycles, a chain of load, compare, branch, select,
  // shuffle and FMA latencies, which is more than the factoring warps need per pivot: the warp with all 32
  // columns to go through finished 1400 cycles after the last pivot and held up the whole block step.
  // The count of columns, 32 - 4 part, is a multiple of four.  A rolled loop: small enough to be served from
  // the innermost instruction cache.
#pragma unroll 1
  for (int k = j0; k < kB; k += 4) {
    uint32_t bits[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      bits[q] = *reinterpret_cast<const volatile uint32_t*>(mcol + (k + q) * kLcolLd + lane);
    float w[4];
#pragma unroll
    for (int q = 0; q < 4; ++q)
      w[q] = (bits[q] != kUnset) ? __uint_as_float(bits[q]) : wait_word(mcol + (k + q) * kLcolLd + lane, gave_up);
    __syncwarp();
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const int kk = k + q;
      my_rinv = (lane == kk) ? w[q] : my_rinv;
      const float m = (lane > kk) ? w[q] : 0.f;
      const float2 nm = make_float2(-m, -m);
      const float2 r01 = make_float2(__shfl_sync(0xffffffffu, x01.x, kk), __shfl_sync(0xffffffffu, x01.y, kk));
      const float2 r23 = make_float2(__shfl_sync(0xffffffffu, x23.x, kk), __shfl_sync(0xffffffffu, x23.y, kk));
      x01 = __ffma2_rn(nm, r01, x01);
      x23 = __ffma2_rn(nm, r23, x23);
    }
  }
  *reinterpret_cast<float4*>(slot + lane * kLd + j0) =
      make_float4(x01.x * my_rinv, x01.y * my_rinv, x23.x * my_rinv, x23.y * my_rinv);
  fence_async_proxy();   // the block is sent on with a bulk copy
  __syncwarp();
}

__global__ void __launch_bounds__(kCThreads, 1) small_block_cluster_kernel(SCParams p) {
  extern __shared__ __align__(16) unsigned char sc_smem[];
  // all barriers complete once; the same layout in every CTA, so a local address maps to any peer
  __shared__ __align__(8) uint64_t dinv_bar[kMaxBlk];    // workers: D_k^{-1} has arrived
  __shared__ __align__(8) uint64_t panel_bar[kMaxBlk];   // workers: every L(i,k), i > k, has arrived
  __shared__ __align__(8) uint64_t chain_bar[kMaxBlk];   // CTA 0: blocks (j, j-1) and (j, j) have arrived
  // workers: L(k+1, k) and L(k+2, k) have arrived -- all that the two blocks CTA 0 waits for next need, so
  // their update does not wait for the whole panel (every worker's blocks, copied to every other worker)
  __shared__ __align__(8) uint64_t urgent_bar[kMaxBlk];
  __shared__ float s_red[kCThreads / 32];
  __shared__ float s_shift, s_floor;
  __shared__ int s_gave_up;
  __shared__ volatile int s_urgent;                       // workers: the factorisation half is on the chain's critical path
  __shared__ volatile int s_chain_step;                   // CTA 0: what the sender warps may send
  __shared__ int s_clamped;
  __shared__ float s_est[kCl];       // CTA 0: the workers' shares of the estimate; workers: per-warp sums
  // blocks (i, j) owned by this CTA, in column-major order
  __shared__ unsigned char s_mine_i[kMaxTri], s_mine_j[kMaxTri];
  __shared__ int s_n_mine;

  float* slots = reinterpret_cast<float*>(sc_smem);        // kMaxTri slots: the matrix, then L / D^{-1}
  float* xt = slots + kMaxTri * kSlot;                      // kXSlots slots: transposed inverse blocks
  float* lcol = xt + kXSlots * kSlot;                       // columns of the diagonal block's factor
  float* mcol = lcol + kB * kLcolLd;                        // the same, scaled by the pivot

  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const int cta = (int)rank;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int r = p.r;
  const int nblk = (r + kB - 1) / kB;
  const int ntri = nblk * (nblk + 1) / 2;

  // A gated launch that is not needed leaves before any set-up: the same word in every CTA of the cluster, written at
  // least two kernels back in the stream (this grid only starts once its predecessor has passed its own
  // griddepcontrol.wait), so it may be read this early.  The wait is still executed: the completion of this grid
  // must imply the completion of every earlier one.
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) { pdl_wait(); pdl_launch_dependents(); return; }

  // ---- set-up, spread over threads: barriers (with the byte counts they will receive, known up front),
  // this CTA's block list, the sentinel words of the diagonal-block column buffer
  if (tid < kMaxBlk) {
    const int k = tid;
    bar_init(&dinv_bar[k], 1);
    bar_init(&panel_bar[k], 2);   // the byte count (below) and the CTA's own blocks of the column
    bar_init(&chain_bar[k], 1);
    bar_init(&urgent_bar[k], 2);  // the byte count, and this CTA's own L(k+2, k) (at once if it owns none)
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (k < nblk) {
      if (cta != 0) {
        bar_expect(&dinv_bar[k], kSlotTx);
        if (k + 1 < nblk) {
          int from_peers = 0;   // rows k + 3 and below; L(k+1, k) (from CTA 0) and L(k+2, k) count on urgent_bar
          for (int bi = k + 3; bi < nblk; ++bi) from_peers += owner_of(bi, k, nblk) != cta ? 1 : 0;
          bar_expect(&panel_bar[k], (uint32_t)from_peers * kSlotTx);
          const bool own_k2 = k + 2 < nblk && owner_of(k + 2, k, nblk) == cta;
          const bool peer_k2 = k + 2 < nblk && !own_k2;
          bar_expect(&urgent_bar[k], (peer_k2 ? 2u : 1u) * kSlotTx);
          if (!own_k2) bar_arrive_local(&urgent_bar[k]);
        }
      } else if (k >= 2) {
        bar_expect(&chain_bar[k], 2 * kSlotTx);
      }
    }
  } else if (tid == 32) {
    s_gave_up = 0;
    s_clamped = 0;
    s_chain_step = 0;
    s_urgent = 0;
    int n = 0;
    for (int bj = 0; bj < nblk; ++bj)
      for (int bi = bj; bi < nblk; ++bi)
        if (owner_of(bi, bj, nblk) == cta) { s_mine_i[n] = (unsigned char)bi; s_mine_j[n] = (unsigned char)bj; ++n; }
    s_n_mine = n;
  }
  for (int e = tid; e < 2 * kB * kLcolLd; e += kCThreads) reinterpret_cast<uint32_t*>(lcol)[e] = kUnset;
  // everything above overlaps the tail of the previous kernel; global memory only from here on
  pdl_wait();
  pdl_launch_dependents();
  // The same word in every CTA, read before anything crosses between them: the whole cluster leaves together.
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) return;

  // ---- load.  Block t is summed over the partials by CTA t mod 8 and written into the slot of the CTA
  // that works on it first (CTA 0 for block rows 0 and 1, the owner otherwise).  All global loads of a
  // thread are issued before the first use; the trace of W (same order of additions in every CTA) gives
  // the diagonal shift and the pivot floor.
  {
    float t = 0.f;
    const int n_scale = p.scale_diag ? p.scale_n : r;
    if (p.scale_diag) {
      for (int i = tid; i < n_scale; i += kCThreads) t += __ldg(p.scale_diag + (int64_t)i * (p.scale_ld + 1));
    } else {
      for (int i = tid; i < r; i += kCThreads) {
        float d = 0.f;
        for (int q = 0; q < p.n_partials; ++q)
          d += __ldg(p.partials + (int64_t)q * p.partial_stride + (int64_t)i * p.in_ld + i);
        t += d;
      }
    }
    constexpr int kMaxMine = (kMaxTri + kCl - 1) / kCl;          // blocks one CTA loads
    constexpr int kPerThread = kMaxMine * (kB * kB / 4) / kCThreads + 1;
    float4 acc[kPerThread];
    const int n_load = (ntri - cta + kCl - 1) / kCl;              // blocks cta, cta + 8, ...
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      acc[u] = make_float4(0.f, 0.f, 0.f, 0.f);
      const int e = tid + u * kCThreads;
      const int lb = e >> 8;                                      // 256 quads per block
      if (lb >= n_load) continue;
      const int blk = cta + lb * kCl;
      int bi = 0;
      while (tri(bi + 1, 0) <= blk) ++bi;
      const int bj = blk - tri(bi, 0);
      const int a = (e & 255) >> 3, q4 = e & 7;
      const int row = bi * kB + a, col = bj * kB + 4 * q4;
      if (row < r && col < r) {
        const float* src = p.partials + (int64_t)row * p.in_ld + col;
        for (int q = 0; q < p.n_partials; ++q) {
          const float4 v = __ldg(reinterpret_cast<const float4*>(src + (int64_t)q * p.partial_stride));
          acc[u].x += v.x; acc[u].y += v.y; acc[u].z += v.z; acc[u].w += v.w;
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (lane == 0) s_red[warp] = t;
    __syncthreads();
    if (tid == 0) {
      float tr = 0.f;
      for (int q = 0; q < kCThreads / 32; ++q) tr += s_red[q];
      float mean_diag = tr / (float)n_scale;
      if (!(mean_diag == mean_diag) || mean_diag > 3.0e38f || mean_diag < 0.f) {
        if (p.dev_status && cta == 0) atomicOr(p.dev_status, LORACT_DEV_NONFINITE);
        mean_diag = 1.f;
      }
      if (mean_diag == 0.f) mean_diag = 1.f;
      s_shift = p.shift_rel * mean_diag;
      s_floor = mean_diag * 1e-7f;
    }
    __syncthreads();
    const float shift = s_shift;
#pragma unroll
    for (int u = 0; u < kPerThread; ++u) {
      const int e = tid + u * kCThreads;
      const int lb = e >> 8;
      if (lb >= n_load) continue;
      const int blk = cta + lb * kCl;
      int bi = 0;
      while (tri(bi + 1, 0) <= blk) ++bi;
      const int bj = blk - tri(bi, 0);
      const int a = (e & 255) >> 3, q4 = e & 7;
      float4 sv = acc[u];
      if (bi == bj) {
        const int dcol = a - 4 * q4;  // position of the diagonal element inside this quad, if any
        const bool in_range = (bi * kB + a) < r;            // padding rows of a ragged last block: identity
        const float mul = in_range ? p.shift_diag_rel : 0.f, add = in_range ? shift : 1.f;
        if (dcol == 0) sv.x += sv.x * mul + add; else if (dcol == 1) sv.y += sv.y * mul + add;
        else if (dcol == 2) sv.z += sv.z * mul + add; else if (dcol == 3) sv.w += sv.w * mul + add;
      }
      const int dst_cta = bi <= 1 ? 0 : owner_of(bi, bj, nblk);
      const uint32_t dst = map_to_cta(smem_addr(slots + blk * kSlot), dst_cta);
      st_cluster_v4(dst + (uint32_t)((a * kLd + 4 * q4) * 4), sv);
    }
  }
  cluster_sync_all();

  if (cta == 0) {
    // =========================================================== pivot chain
    // Phase A: warps 0, 1 factor the diagonal block, warps 2..9 invert it alongside, a thread of warp 10
    // waits for the two blocks of the next step.  Phase B (warps 0..7): L(k+1, k).  Phase C (warps 0..7):
    // the next diagonal block.  Warp 11 only sends: D_k^{-1} after phase A, L(k+1, k) after phase B; it
    // follows a step counter in shared memory and never holds the others up.
    constexpr int kChainWarps = 11;   // warps that take part in the phase barriers
    if (warp < kChainWarps) {
      for (int k = 0; k < nblk; ++k) {
        float* dslot = slots + tri(k, k) * kSlot;
        if (warp < 2) {
          if (factor_diag_half(dslot, lcol, mcol, s_floor, &s_gave_up, warp, lane) && lane == 0) s_clamped = 1;
        } else if (warp < 2 + kInvWarps) {
          invert_diag_part(dslot, mcol, &s_gave_up, warp - 2, lane);
        } else if (lane == 0 && k + 1 < nblk && k >= 1) {
          bar_wait(&chain_bar[k + 1], &s_gave_up);   // blocks (k+1, k) and (k+1, k+1)
        }
        chain_sync();
        if (tid == 0) { __threadfence_block(); s_chain_step = 2 * k + 1; }
        if (k + 1 >= nblk) break;
        // L(k+1, k) = A(k+1, k) D_k^{-T}, in place (a warp reads only the rows it writes)
        float* sub = slots + tri(k + 1, k) * kSlot;
        if (warp < 8) {
          float acc[2][2];
          tile_zero(acc);
          tile_mac<2, 2>(acc, sub, dslot, tid >> 4, tid & 15);
          group_sync(1);   // in place: everyone has read the block
          tile_store<2, 2>(sub, acc, tid >> 4, tid & 15, 1.f, false);
          fence_async_proxy();   // the block is sent on with a bulk copy
        }
        chain_sync();
        if (tid == 0) { __threadfence_block(); s_chain_step = 2 * k + 2; }
        if (warp < 8) {
          // next diagonal block: A(k+1, k+1) -= L(k+1, k) L(k+1, k)^T
          float acc2[2][2];
          tile_zero(acc2);
          tile_mac<2, 2>(acc2, sub, sub, tid >> 4, tid & 15);
          tile_store<2, 2>(slots + tri(k + 1, k + 1) * kSlot, acc2, tid >> 4, tid & 15, -1.f, true);
        } else {
          for (int e = tid - 8 * 32; e < 2 * kB * kLcolLd; e += (kChainWarps - 8) * 32)
            reinterpret_cast<uint32_t*>(lcol)[e] = kUnset;
        }
        chain_sync();
      }
      if (tid == 0 && s_clamped && p.dev_status) atomicOr(p.dev_status, LORACT_DEV_PIVOT_CLAMPED);
    } else if (warp == kChainWarps) {
      // the sender: lane c copies each finished block to CTA c
      for (int step = 1; step <= 2 * nblk - 1; ++step) {
        // step 2k + 1: D_k^{-1} is ready;  step 2k + 2: L(k+1, k) is ready
        if (lane == 0) {
          uint64_t t0 = 0;
          for (uint32_t spin = 1; s_chain_step < step; ++spin) {
            __nanosleep(20);
            if ((spin & 255u) == 0u) {
              if (*(volatile int*)&s_gave_up) break;
              const uint64_t now = timer_ns();
              if (t0 == 0) t0 = now;
              else if (now - t0 > kClusterWaitNs) { s_gave_up = 1; break; }
            }
          }
          __threadfence_block();
        }
        __syncwarp();
        const int k = (step - 1) >> 1;
        const bool is_dinv = (step & 1) != 0;
        const float* blk = slots + (is_dinv ? tri(k, k) : tri(k + 1, k)) * kSlot;
        if (lane >= 1 && lane < kCl) {
          const uint32_t src = smem_addr(blk);
          bulk_to_peer(map_to_cta(src, lane), src, kSlotTx,
                       map_to_cta(smem_addr(is_dinv ? &dinv_bar[k] : &urgent_bar[k]), lane));
        }
      }
    }
  } else if (warp < 8) {
    // =========================================================== workers, factorisation half
    // Four pairs of warps; a pair does one 32 x 32 block product at a time (4 x 4 outputs per thread), the
    // blocks of a phase are dealt out to the pairs in turn.  Warp h of a pair holds rows 16 h .. 16 h + 15.
    const int pair = warp >> 1;
    const int tp = tid & 63, tm = tp >> 3, tn = tp & 7;   // 4 x 4 outputs per thread on a pair of warps
    const int t2m = tid >> 4, t2n = tid & 15;             // 2 x 2 outputs per thread on all eight warps
    const int n_mine = s_n_mine;
    for (int k = 0; k < nblk; ++k) {
      if (tid == 0) {
        bar_wait(&dinv_bar[k], &s_gave_up);
        s_urgent = 1;   // the other half of the CTA stands back until the chain has what it waits for
      }
      group_sync(1);
      const float* dk = slots + tri(k, k) * kSlot;
      // L(i, k) = A(i, k) D_k^{-T} for the block of column k this CTA owns (CTA 0 does block k + 1): on the
      // critical path, so all eight warps share the one product; in place
      for (int q = 0; q < n_mine; ++q) {
        const int bi = s_mine_i[q], bj = s_mine_j[q];
        if (bj != k || bi < k + 2) continue;
        float* blk = slots + tri(bi, k) * kSlot;
        float acc[2][2];
        tile_zero(acc);
        tile_mac<2, 2>(acc, blk, dk, t2m, t2n);
        group_sync(1);   // everyone has read the block
        tile_store<2, 2>(blk, acc, t2m, t2n, 1.f, false);
        fence_async_proxy();
        send_rows(blk, warp * 4, 4, bi == k + 2 ? &urgent_bar[k] : &panel_bar[k], 1, kCl - 1, cta, lane);
      }
      // this CTA's own blocks of column k are in place: the second arrival on its own barriers
      group_sync(1);
      if (tid == 0 && k + 1 < nblk) {
        bar_arrive_local(&panel_bar[k]);
        if (k + 2 < nblk && owner_of(k + 2, k, nblk) == cta) bar_arrive_local(&urgent_bar[k]);
      }
      if (k + 1 >= nblk) { if (tid == 0) s_urgent = 0; break; }
      if (tid == 0) bar_wait(&urgent_bar[k], &s_gave_up);
      group_sync(1);
      // trailing update with column k.  A diagonal block (j, j) takes columns k <= j - 2 here (CTA 0
      // applies column j - 1 itself), every other block (i, j) columns k <= j - 1.  First the two blocks
      // CTA 0 needs next, each on all eight warps, sent on as soon as they are done ...
      for (int q = 0; q < n_mine; ++q) {
        const int bi = s_mine_i[q], bj = s_mine_j[q];
        if (bi != k + 2 || (bj != k + 1 && bj != k + 2)) continue;
        float acc[2][2];
        tile_zero(acc);
        tile_mac<2, 2>(acc, slots + tri(bi, k) * kSlot, slots + tri(bj, k) * kSlot, t2m, t2n);
        float* blk = slots + tri(bi, bj) * kSlot;
        tile_store<2, 2>(blk, acc, t2m, t2n, -1.f, true);
        fence_async_proxy();
        send_rows(blk, warp * 4, 4, &chain_bar[k + 2], 0, 0, -1, lane);
      }
      if (tid == 0) { s_urgent = 0; bar_wait(&panel_bar[k], &s_gave_up); }
      group_sync(1);
      // ... then the rest, one block per pair of warps at a time
      int turn = 0;
      for (int q = 0; q < n_mine; ++q) {
        const int bi = s_mine_i[q], bj = s_mine_j[q];
        if (bi < 2) continue;
        const bool active = (bi == bj) ? (k <= bj - 2) : (k <= bj - 1);
        if (!active) continue;
        if ((bi == k + 2) && (bj == k + 1 || bj == k + 2)) continue;
        if ((turn++ & 3) != pair) continue;
        float acc[4][4];
        tile_zero(acc);
        tile_mac<4, 4>(acc, slots + tri(bi, k) * kSlot, slots + tri(bj, k) * kSlot, tm, tn);
        tile_store<4, 4>(slots + tri(bi, bj) * kSlot, acc, tm, tn, -1.f, true);
      }
    }
  } else {
    // =========================================================== workers, inverse half (warps 8..15)
    // Right-looking by block rows, in transposed storage Xt(i,j)[b][a] = X(i,j)[a][b]: at step k block row
    // k of the inverse becomes final, X(k,j) = -D_k^{-1} T(k,j) (X(k,k) = D_k^{-1}), is written out, and is
    // added into the sums of all later rows, T(i,j) += L(i,k) X(k,j).  Finishing a block is one product on
    // all eight warps (2 x 2 outputs per thread); the products into the later rows are dealt out to four
    // pairs of warps (4 x 4 outputs per thread).
    const int gt = tid - kGroup;
    const int pair = (warp - 8) >> 1;
    const int tp = gt & 63, tm = tp >> 3, tn = tp & 7;
    const int t2m = gt >> 4, t2n = gt & 15;
    // block columns of the inverse this CTA computes: j0 = cta - 1, and 7 as well on the last worker
    const int j0 = cta - 1;
    const int n_cols = (j0 < nblk ? 1 : 0) + ((cta == kWorkers && kWorkers < nblk) ? 1 : 0);
    // for the estimate: the diagonal entries (as factored) of the one or two columns this thread writes
    float wdiag[2] = {0.f, 0.f};
    float est_acc = 0.f;
    if (p.gate_out) {
      for (int cidx = 0; cidx < n_cols; ++cidx) {
        const int col = (j0 + cidx) * kB + (gt & 31);
        if (col < r) {
          float dsum = 0.f;
          for (int q = 0; q < p.n_partials; ++q)
            dsum += __ldg(p.partials + (int64_t)q * p.partial_stride + (int64_t)col * p.in_ld + col);
          wdiag[cidx] = dsum + dsum * p.shift_diag_rel + s_shift;
        }
      }
    }
    // zeros above the diagonal blocks
    for (int cidx = 0; cidx < n_cols; ++cidx) {
      const int j = j0 + cidx;
      const int ncol = min(kB, r - j * kB);
      for (int e = gt; e < j * kB * kB; e += kGroup) {
        const int row = e >> 5, b = e & 31;
        if (b >= ncol) continue;
        const int64_t off = (int64_t)row * p.out_ld + j * kB + b;
        if (p.linv_f32) p.linv_f32[off] = 0.f;
        if (p.linv_hi) p.linv_hi[off] = __float2bfloat16(0.f);
        if (p.linv_lo) p.linv_lo[off] = __float2bfloat16(0.f);
      }
    }
    for (int k = 0; k < nblk; ++k) {
      if (gt == 0) bar_wait(&dinv_bar[k], &s_gave_up);
      group_sync(2);
      const float* dk = slots + tri(k, k) * kSlot;
      for (int cidx = 0; cidx < n_cols; ++cidx) {
        const int j = j0 + cidx;
        if (j > k) continue;
        float* dst = xt + ((cidx == 0 ? 0 : (nblk - j0)) + (k - j)) * kSlot;
        if (j == k) {
          for (int e = gt; e < kB * kB; e += kGroup) {
            const int b = e >> 5, a = e & 31;
            dst[b * kLd + a] = dk[a * kLd + b];
          }
        } else {
          // Xt(k,j)[b][a] = -sum_q Tt(k,j)[b][q] D_k^{-1}[a][q], in place
          float acc[2][2];
          tile_zero(acc);
          tile_mac<2, 2>(acc, dst, dk, t2m, t2n);
          group_sync(2);   // everyone has read the sums
          tile_store<2, 2>(dst, acc, t2m, t2n, -1.f, false);
        }
      }
      group_sync(2);
      // block row k of the result: Linv[k*32 + a][j*32 + b] = Xt(k,j)[b][a]
      for (int cidx = 0; cidx < n_cols; ++cidx) {
        const int j = j0 + cidx;
        if (j > k) continue;
        const float* src = xt + ((cidx == 0 ? 0 : (nblk - j0)) + (k - j)) * kSlot;
        const int ncol = min(kB, r - j * kB);
        for (int e = gt; e < kB * kB; e += kGroup) {
          const int a = e >> 5, b = e & 31;
          const int row = k * kB + a;
          if (row >= r || b >= ncol) continue;
          const float v = src[b * kLd + a];
          est_acc = fmaf(v * v, wdiag[cidx], est_acc);
          const int64_t off = (int64_t)row * p.out_ld + j * kB + b;
          if (p.linv_f32) p.linv_f32[off] = v;
          if (p.linv_hi) {
            const __nv_bfloat16 hi = __float2bfloat16(v);
            p.linv_hi[off] = hi;
            if (p.linv_lo) p.linv_lo[off] = __float2bfloat16(v - __bfloat162float(hi));
          }
        }
      }
      if (k + 1 >= nblk) break;
      if (gt == 0) { bar_wait(&urgent_bar[k], &s_gave_up); bar_wait(&panel_bar[k], &s_gave_up); }
      group_sync(2);
      // Tt(i,j)[b][a] (+)= sum_q Xt(k,j)[b][q] L(i,k)[a][q] for the rows below
      int turn = 0;
      for (int cidx = 0; cidx < n_cols; ++cidx) {
        const int j = j0 + cidx;
        if (j > k) continue;
        float* xcol = xt + (cidx == 0 ? 0 : (nblk - j0)) * kSlot;   // block (i, j) at xcol + (i - j) slots
        const float* xk = xcol + (k - j) * kSlot;
        for (int i = k + 1; i < nblk; ++i) {
          if ((turn++ & 3) != pair) continue;
          for (int spin = 0; s_urgent && spin < 256; ++spin) __nanosleep(64);   // a hint, not a lock
          float acc[4][4];
          tile_zero(acc);
          tile_mac<4, 4>(acc, xk, slots + tri(i, k) * kSlot, tm, tn);
          tile_store<4, 4>(xcol + (i - j) * kSlot, acc, tm, tn, 1.f, j != k);
        }
      }
    }
    if (p.gate_out) {
      // this CTA's share of the estimate, summed in a fixed order and handed to CTA 0
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) est_acc += __shfl_xor_sync(0xffffffffu, est_acc, o);
      if (lane == 0) s_est[warp - 8] = est_acc;
      group_sync(2);
      if (gt == 0) {
        float t = 0.f;
        for (int q = 0; q < 8; ++q) t += s_est[q];
        asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(map_to_cta(smem_addr(&s_est[cta]), 0)), "f"(t) : "memory");
      }
    }
  }
  __syncthreads();
  if (tid == 0 && s_gave_up && p.dev_status) atomicOr(p.dev_status, LORACT_DEV_WAIT_EXPIRED);
  // no CTA leaves while another may still write into its shared memory
  cluster_sync_all();
  if (p.gate_out && cta == 0 && tid == 0) {
    // after the cluster barrier: every worker's share has arrived, every status bit of this call is set
    float est = 0.f;
    for (int c = 1; c < kCl; ++c) est += s_est[c];
    const uint32_t st = p.dev_status ? atomicOr(p.dev_status, 0u) : 0u;
    const bool again = !(est <= p.gate_threshold) || st != 0u;
    p.gate_out[0] = again ? 1u : 0u;
    p.gate_out[1] = __float_as_uint(est);
    p.gate_out[2] = again ? 2u : 1u;
  }
}

// The give-up path of this file's waits, exercised on purpose: a two-CTA cluster in which CTA 1 waits, with
// bar_wait, for bytes that CTA 0 never sends.  After `limit_ns` it records LORACT_DEV_WAIT_EXPIRED and both
// CTAs run to the closing cluster barrier, as the factorisation kernel does.
__global__ void __cluster_dims__(2, 1, 1) cluster_wait_probe_kernel(uint32_t* dev_status, uint64_t limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int gave_up;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  if (threadIdx.x == 0) {
    bar_init(&bar, 1);
    gave_up = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    bar_expect(&bar, 16);   // sixteen bytes that never arrive
  }
  cluster_sync_all();
  if (rank == 1 && threadIdx.x == 0) bar_wait(&bar, &gave_up, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && gave_up && dev_status) atomicOr(dev_status, LORACT_DEV_WAIT_EXPIRED);
  cluster_sync_all();
}

}  // namespace

cudaError_t small_block_cluster_wait_probe_launch(uint32_t* dev_status, uint64_t limit_ns, cudaStream_t stream) {
  cluster_wait_probe_kernel<<<2, 32, 0, stream>>>(dev_status, limit_ns);
  count_launch(__func__, stream);
  return cudaGetLastError();
}

bool small_block_cluster_supported(const SmallBlockArgs& a) {
  return !a.use_f64 && a.partial_type == ELEM_F32 && a.r <= kMaxBlk * kB && a.r % 4 == 0 &&
         a.linv_full == nullptr && (((uintptr_t)a.partials & 15) == 0) && (a.partial_stride % 4 == 0) && (a.in_ld % 4 == 0);
}

cudaError_t small_block_cluster_launch(const SmallBlockArgs& a, cudaStream_t stream) {
  SCParams p;
  p.r = a.r;
  p.partials = (const float*)a.partials;
  p.in_ld = a.in_ld ? a.in_ld : a.r;
  p.out_ld = a.out_ld ? a.out_ld : a.r;
  p.n_partials = a.n_partials;
  p.partial_stride = a.partial_stride;
  p.shift_rel = a.shift_rel;
  p.shift_diag_rel = a.shift_diag_rel;
  p.gate = a.gate;
  p.gate_out = a.gate_out;
  p.gate_threshold = a.gate_threshold;
  p.linv_f32 = a.linv_f32;
  p.linv_hi = a.linv_hi;
  p.linv_lo = a.linv_lo;
  p.dev_status = a.dev_status;
  p.scale_diag = a.scale_diag;
  p.scale_n = a.scale_n;
  p.scale_ld = a.scale_ld;
  const size_t smem = (size_t)(kMaxTri + kXSlots) * kSlot * sizeof(float) + (size_t)(2 * kB * kLcolLd) * sizeof(float);
  static std::atomic<bool> configured[64];
  int dev = 0;
  LORACT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    LORACT_CUDA_TRY(cudaFuncSetAttribute(small_block_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)smem));
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(kCl, 1, 1);
  cfg.blockDim = dim3(kCThreads, 1, 1);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = kCl;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  LORACT_CUDA_TRY(cudaLaunchKernelEx(&cfg, small_block_cluster_kernel, p));
  count_launch();
  return cudaGetLastError();
}

}  // namespace loract

// Tensor-core engine for the dense contractions of the path (the sketch and the projection of Algorithm 1, the Gram
// matrices of the orthonormalisation, the application of the triangular factors, Reconstruct).
//
// One kernel, written for sm_100a: TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) fills a
// 4-stage shared-memory ring, one thread issues tcgen05.mma (kind::f16, bf16 operands, M = 128,
// N <= 256, K = 16 per instruction) into an fp32 accumulator in tensor memory, four warps read the
// accumulator back with tcgen05.ld and write the result.  Operands may be K-major or MN-major, which
// covers X Omega^T (K/K), U^T X and Y^T Y (MN/MN) and U V (K/MN) without transposing anything in memory.
// A contraction can be the sum of up to three products over the same shapes (split-precision terms),
// and can be split over K into partial results that a later kernel adds in a fixed order.
//
// Every wait on an mbarrier is bounded by a wall-clock limit; on expiry the kernel records
// LORACT_DEV_WAIT_EXPIRED, stops issuing work, frees its tensor memory and returns.
#include <cuda.h>

#include <map>
#include <atomic>
#include <mutex>
#include <tuple>

#include "common.cuh"

namespace loract {

namespace {

constexpr int kBM = 128;
constexpr int kBK = 64;          // bf16 elements = one 128-byte swizzle row
constexpr int kStages = 4;
constexpr int kThreads = 320;    // warp 0: TMA, warp 1: MMA + tensor memory, warps 2..9: epilogue
constexpr int kEpiWarps = 8;     // two per quarter of the tensor-memory lanes: they take alternate column groups
constexpr uint32_t kABytes = kBM * kBK * 2;
constexpr uint64_t kWaitLimitNs = 2000000000ull;  // 2 s

struct alignas(64) TmapPack {
  CUtensorMap a[3];
  CUtensorMap b[3];
  CUtensorMap c[2];   // outputs (C0, C1) for the staged epilogue: boxes of 128 bytes x 32 rows
};

struct TcParams {
  int M, N;
  int bn;             // tile width, multiple of 16, <= 256
  int kb_total;       // 64-wide K blocks per term
  int kb_per_split;
  int n_terms;
  int out;
  void* C0;
  void* C1;
  int64_t ldc;
  int64_t split_stride;
  uint32_t b_bytes;   // bytes of one B stage
  uint32_t tmem_cols;
  int accumulate;     // OUT_F32, one split: C += result
  const void* ep_E;   // OUT_RMS_BWD epilogue operands
  int64_t ep_ld;
  const float* ep_row_a;
  const float* ep_row_b;
  const void* ep_col;
  int ep_kind;        // OUT_ACT_BWD: 0 SiLU, 1 GELU
  uint32_t* dev_status;
  int tma_store;      // 1: the epilogue stages 32-row boxes in shared memory and writes them with TMA stores
  int st_m_tiles;     // streaming kernel: 256-row tiles along M
  int st_units;       // streaming kernel: tiles in all (column tile major, then M)
  int st_stages;      // streaming kernel: stages of the A ring (<= kStreamStages)
  int store_bufs;     // staging boxes per epilogue warp (1 or 2)
  int halve_at_term;  // the accumulator is multiplied by 1/2 before the first product of this term (0: never)
  int a_keep_from_kb; // two-CTA kernel: K block from which the loads of A carry an evict-last hint (kb_total: none)
  // one-tile kernels: when set and the word it points to is zero, the kernel loads, multiplies and stores nothing
  // (a step that an earlier kernel of the same stream found unnecessary)
  const uint32_t* gate;
  // one-tile kernels: block (0, 0, 0) stores zero into *dev_status right after griddepcontrol.wait (for the first
  // kernel of a call: no memset node in front of the chain).  A bounded wait of this kernel can set a bit two seconds
  // later at the earliest, long after that store.
  int clear_status;
  // one-tile kernels, OUT_SPLIT: when set and the word is zero, the low part (C1) is not written
  const uint32_t* lo_gate;
};

// ------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ uint64_t global_timer_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait.  Returns false if the limit expired (or another role already gave up).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag,
                                                  uint64_t limit_ns = kWaitLimitNs) {
  if (mbar_try_wait(bar, parity)) return true;
  // the wall clock is read only once in a while, and first after 1024 failed polls: a read of %globaltimer is
  // slow enough to matter on the hand-offs of the operand ring, which all pass through here
  uint64_t t0 = 0;
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((spin & 1023u) == 0u) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > limit_ns) { *abort_flag = 1; return false; }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(void* smem_dst, const CUtensorMap* map, uint64_t* bar, int x,
                                            int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)map), "r"(smem_u32(bar)), "r"(x), "r"(y)
      : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_mma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                            uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// The same instruction with the accumulator read as D / 2 (scale-input-d = 1): D = A B + D * 2^-1.
__device__ __forceinline__ void tc_mma_bf16_halved(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, 1, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p, 1;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
      : "memory");
}
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t v[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_ld64(uint32_t taddr, uint32_t v[64]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31]), "=r"(v[32]), "=r"(v[33]), "=r"(v[34]), "=r"(v[35]), "=r"(v[36]), "=r"(v[37]), "=r"(v[38]), "=r"(v[39]), "=r"(v[40]), "=r"(v[41]), "=r"(v[42]), "=r"(v[43]), "=r"(v[44]), "=r"(v[45]), "=r"(v[46]), "=r"(v[47]), "=r"(v[48]), "=r"(v[49]), "=r"(v[50]), "=r"(v[51]), "=r"(v[52]), "=r"(v[53]), "=r"(v[54]), "=r"(v[55]), "=r"(v[56]), "=r"(v[57]), "=r"(v[58]), "=r"(v[59]), "=r"(v[60]), "=r"(v[61]), "=r"(v[62]), "=r"(v[63])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tc_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Shared-memory matrix descriptor, 128-byte swizzle.  K-major: rows of 128 bytes, groups of 8 rows
// 1024 bytes apart (stride byte offset); the leading byte offset is not used.  MN-major: rows are K
// indices, each 128 bytes = 64 elements along M/N; groups of 8 K rows 1024 bytes apart (stride byte
// offset) and consecutive 64-element groups along M/N one TMA box (64 rows = 8192 bytes) apart
// (leading byte offset).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t smem_addr, bool mn_major) {
  const uint64_t lbo = mn_major ? (8192u >> 4) : 1u;
  const uint64_t sbo = 1024u >> 4;
  return (uint64_t)((smem_addr >> 4) & 0x3FFFu) | (lbo << 16) | (sbo << 32) | (1ull << 46) | (2ull << 61);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 t = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&t);
}

// f'(a) of the element-wise consumers (OUT_ACT_BWD).  SiLU: s (1 + a (1 - s)), s the logistic function;
// GELU (exact form): Phi(a) + a phi(a).  The result is multiplied by the upstream gradient and rounded to bf16.
__device__ __forceinline__ float act_derivative(float a, int kind) {
  if (kind == 0) {
    const float s = 1.f / (1.f + __expf(-a));
    return s * (1.f + a * (1.f - s));
  }
  return 0.5f * (1.f + erff(a * 0.70710678118f)) + a * 0.39894228040f * __expf(-0.5f * a * a);
}

// ---- staged epilogue.  A thread owns one accumulator row, so a direct store instruction of a warp touches 32
// different rows, 16 bytes each: every 128-byte line of the output is written in eight pieces by eight
// instructions.  Instead each epilogue warp puts its 32 rows x 128 bytes into shared memory in the layout of a
// 128-byte-swizzled TMA box (conflict free: the 16-byte chunk c of row i goes to chunk c ^ (i & 7)) and one
// lane sends the box with a TMA store, which writes whole lines and clips at the edges of the output.  Each
// warp cycles through kStoreBufs boxes of its own, so no barrier between warps is needed.  Two warps share each
// quarter of the accumulator rows (a warp may only read the tensor-memory lanes 32 * (warp % 4) .. + 31); they
// take alternate column groups.
constexpr int kStoreBufs = 2;
constexpr uint32_t kStoreBoxBytes = 4096;                    // 32 rows x 128 bytes
constexpr uint32_t kStoreWarpBytes = kStoreBufs * kStoreBoxBytes;

struct StoreStage {
  unsigned char* base;   // this warp's boxes (1024-byte aligned); nullptr: direct stores only
  uint32_t cnt;          // boxes sent so far
  uint32_t bufs;         // boxes this warp cycles through (1 or 2)
};

__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, const void* smem_src, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"((uint64_t)map), "r"(smem_u32(smem_src)), "r"(x), "r"(y)
               : "memory");
}
template <int kPending>
__device__ __forceinline__ void bulk_wait_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(kPending) : "memory");
}
// Boxes cnt .. cnt + kNeed - 1 may be written once the stores that last used them have read shared memory.
template <int kNeed>
__device__ __forceinline__ void stage_acquire(const StoreStage& st, int lane) {
  if (st.cnt + kNeed > st.bufs) {
    if (lane == 0) {
      if (st.bufs > (uint32_t)kNeed) bulk_wait_read<kStoreBufs - kNeed>();
      else bulk_wait_read<0>();
    }
    __syncwarp();
  }
}
__device__ __forceinline__ unsigned char* stage_box(const StoreStage& st, uint32_t k) {
  return st.base + (st.bufs == 1 ? 0u : ((st.cnt + k) & 1u)) * kStoreBoxBytes;
}
__device__ __forceinline__ void stage_write16(unsigned char* box, int lane, int chunk, uint4 v) {
  *reinterpret_cast<uint4*>(box + lane * 128 + ((chunk ^ (lane & 7)) << 4)) = v;
}
// All lanes have written their rows of `box`: make them visible to the async proxy and send the box.
__device__ __forceinline__ void stage_send(const CUtensorMap* map, unsigned char* box, int lane, int x, int y) {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  __syncwarp();
  if (lane == 0) {
    tma_store_2d(map, box, x, y);
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
  }
}
// Before the shared memory goes away (or at the end of the kernel): every store of this warp is complete.
__device__ __forceinline__ void stage_drain(const StoreStage& st, int lane) {
  if (st.base && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  __syncwarp();
}

__device__ __forceinline__ void tc_store_tile_staged(const TcParams& p, const TmapPack& maps, uint32_t tmem_base,
                                                     int quad, int half_id, int lane, int m0, int n0,
                                                     int split, StoreStage& st, bool lo_on = true) {
  const int row0 = m0 + quad * 32;
  const int m = row0 + lane;
  const uint32_t taddr = tmem_base + ((uint32_t)(quad * 32) << 16);
  const int y = split * p.M + row0;
  if (p.out == OUT_F32) {
    for (int c0 = 32 * half_id; c0 < p.bn && n0 + c0 < p.N; c0 += 64) {
      uint32_t v[32];
      tc_ld32(taddr + (uint32_t)c0, v);
      tc_wait_ld();
      stage_acquire<1>(st, lane);
      unsigned char* box = stage_box(st, 0);
#pragma unroll
      for (int q = 0; q < 8; ++q) stage_write16(box, lane, q, make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]));
      stage_send(&maps.c[0], box, lane, n0 + c0, y);
      st.cnt += 1;
    }
    return;
  }
  const bool split_out = p.out == OUT_SPLIT && lo_on;   // lo_on false: only the leading part is wanted
  const bool rms = p.out == OUT_RMS_BWD;
  const bool act = p.out == OUT_ACT_BWD;
  const bool live = m < p.M;                                 // rows past M are clipped by the store
  float ra = 0.f, rb = 0.f;
  if (rms && live) { ra = p.ep_row_a[m]; rb = p.ep_row_b[m]; }
  for (int c0 = 64 * half_id; c0 < p.bn && n0 + c0 < p.N; c0 += 128) {
    if (split_out) stage_acquire<2>(st, lane); else stage_acquire<1>(st, lane);
    unsigned char* box_hi = stage_box(st, 0);
    unsigned char* box_lo = stage_box(st, 1);
    uint32_t v64[64];
    tc_ld64(taddr + (uint32_t)c0, v64);
    tc_wait_ld();
#pragma unroll
    for (int half = 0; half < 2; ++half) {
      const uint32_t* v = v64 + 32 * half;
      const int n = n0 + c0 + 32 * half;
      if (rms) {
        const bool cols_ok = n + 32 <= p.N;                  // a partial group is clipped anyway; read nothing past N
        const __nv_bfloat16* e = (const __nv_bfloat16*)p.ep_E + (int64_t)m * p.ep_ld + n;
        const __nv_bfloat16* col = (const __nv_bfloat16*)p.ep_col + n;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t ow[4] = {0u, 0u, 0u, 0u};
          if (live && cols_ok) {
            const uint4 ev = reinterpret_cast<const uint4*>(e)[q];
            const uint4 cv = __ldg(reinterpret_cast<const uint4*>(col) + q);
            const uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w}, cw[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              const float e0 = __uint_as_float(ew[h] << 16), e1 = __uint_as_float(ew[h] & 0xffff0000u);
              const float c0f = __uint_as_float(cw[h] << 16), c1f = __uint_as_float(cw[h] & 0xffff0000u);
              const float a0 = __uint_as_float(v[8 * q + 2 * h]), a1 = __uint_as_float(v[8 * q + 2 * h + 1]);
              // the quotient is rounded to bf16 below: the fast division (2 ulp in fp32) is exact enough
              ow[h] = pack_bf16x2(ra * c0f * e0 - __fdividef(rb * a0, c0f), ra * c1f * e1 - __fdividef(rb * a1, c1f));
            }
          } else if (live) {
            for (int h = 0; h < 8; ++h) {
              const int nn = n + 8 * q + h;
              if (nn < p.N) {
                const float c = __bfloat162float(col[8 * q + h]);
                const float r = ra * c * __bfloat162float(e[8 * q + h]) - rb * __uint_as_float(v[8 * q + h]) / c;
                const uint32_t bits = (uint32_t)__bfloat16_as_ushort(__float2bfloat16(r));
                ow[h >> 1] |= (h & 1) ? (bits << 16) : bits;
              }
            }
          }
          stage_write16(box_hi, lane, 4 * half + q, make_uint4(ow[0], ow[1], ow[2], ow[3]));
        }
      } else if (act) {
        const bool cols_ok = n + 32 <= p.N;
        const __nv_bfloat16* e = (const __nv_bfloat16*)p.ep_E + (int64_t)m * p.ep_ld + n;
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t ow[4] = {0u, 0u, 0u, 0u};
          if (live && cols_ok) {
            const uint4 ev = reinterpret_cast<const uint4*>(e)[q];
            const uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w};
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              const float e0 = __uint_as_float(ew[h] << 16), e1 = __uint_as_float(ew[h] & 0xffff0000u);
              const float a0 = __uint_as_float(v[8 * q + 2 * h]), a1 = __uint_as_float(v[8 * q + 2 * h + 1]);
              ow[h] = pack_bf16x2(e0 * act_derivative(a0, p.ep_kind), e1 * act_derivative(a1, p.ep_kind));
            }
          } else if (live) {
            for (int h = 0; h < 8; ++h) {
              const int nn = n + 8 * q + h;
              if (nn < p.N) {
                const float r = __bfloat162float(e[8 * q + h]) * act_derivative(__uint_as_float(v[8 * q + h]), p.ep_kind);
                const uint32_t bits = (uint32_t)__bfloat16_as_ushort(__float2bfloat16(r));
                ow[h >> 1] |= (h & 1) ? (bits << 16) : bits;
              }
            }
          }
          stage_write16(box_hi, lane, 4 * half + q, make_uint4(ow[0], ow[1], ow[2], ow[3]));
        }
      } else if (!split_out) {
        // one conversion instruction per pair of columns: this loop runs on a single warp per scheduler, so
        // its length in instructions is its duration
#pragma unroll
        for (int q = 0; q < 4; ++q)
          stage_write16(box_hi, lane, 4 * half + q,
                        make_uint4(pack_bf16x2(__uint_as_float(v[8 * q]), __uint_as_float(v[8 * q + 1])),
                                   pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                                   pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                                   pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7]))));
      } else {
        uint32_t hi[16], lo[16];
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          const float x0 = __uint_as_float(v[2 * q]), x1 = __uint_as_float(v[2 * q + 1]);
          hi[q] = pack_bf16x2(x0, x1);
          lo[q] = pack_bf16x2(x0 - __uint_as_float(hi[q] << 16), x1 - __uint_as_float(hi[q] & 0xffff0000u));
        }
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          stage_write16(box_hi, lane, 4 * half + q, make_uint4(hi[4 * q], hi[4 * q + 1], hi[4 * q + 2], hi[4 * q + 3]));
          stage_write16(box_lo, lane, 4 * half + q, make_uint4(lo[4 * q], lo[4 * q + 1], lo[4 * q + 2], lo[4 * q + 3]));
        }
      }
    }
    stage_send(&maps.c[0], box_hi, lane, n0 + c0, y);
    if (split_out) stage_send(&maps.c[1], box_lo, lane, n0 + c0, y);
    st.cnt += split_out ? 2 : 1;
  }
}

// Writes one finished accumulator tile (128 rows of this CTA x bn columns, starting at tensor-memory column
// tmem_base) in the output mode of p.  Warp w may touch the lanes 32 * (w % 4) .. + 31.
__device__ __forceinline__ void tc_store_tile(const TcParams& p, const TmapPack& maps, uint32_t tmem_base, int warp,
                                              int lane, int m0, int n0, int split, StoreStage& st, bool lo_on = true) {
  const int quad = warp & 3;
  const int half_id = (warp - 2) >> 2;                       // which of the two warps of this quarter
  const int row = quad * 32 + lane;
  const int m = m0 + row;
  if (m0 + quad * 32 >= p.M) return;                         // none of this warp's rows exists
  // staged unless the output needs read-modify-write, or (split-K partials stacked along the rows of one
  // tensor map) the warp's 32 rows are not all inside M
  if (st.base && p.tma_store && !p.accumulate && (p.split_stride == 0 || m0 + quad * 32 + 32 <= p.M)) {
    tc_store_tile_staged(p, maps, tmem_base, quad, half_id, lane, m0, n0, split, st, lo_on);
    return;
  }
  {
    for (int c0 = 32 * half_id; c0 < p.bn; c0 += 64) {
      uint32_t v[32];
      tc_ld32(tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)c0, v);
      tc_wait_ld();
      const int n = n0 + c0;
      if (m >= p.M) continue;
      const int valid = min(32, min(p.bn - c0, p.N - n));
      if (valid <= 0) continue;
      if (p.out == OUT_F32) {
        float* dst = (float*)p.C0 + (int64_t)split * p.split_stride + (int64_t)m * p.ldc + n;
        if (p.accumulate) {
          for (int q = 0; q < valid; ++q) dst[q] += __uint_as_float(v[q]);
        } else if (valid == 32 && ((((uintptr_t)dst) & 15) == 0)) {
#pragma unroll
          for (int q = 0; q < 8; ++q)
            reinterpret_cast<uint4*>(dst)[q] = make_uint4(v[4 * q], v[4 * q + 1], v[4 * q + 2], v[4 * q + 3]);
        } else {
          for (int q = 0; q < valid; ++q) dst[q] = __uint_as_float(v[q]);
        }
      } else if (p.out == OUT_RMS_BWD) {
        // grad_X = rstd * (grad_A * gamma - (reconstructed A / gamma) * inner): the tile of the reconstructed
        // activation exists only in tensor memory and in these registers
        __nv_bfloat16* dst = (__nv_bfloat16*)p.C0 + (int64_t)m * p.ldc + n;
        const __nv_bfloat16* e = (const __nv_bfloat16*)p.ep_E + (int64_t)m * p.ep_ld + n;
        const __nv_bfloat16* col = (const __nv_bfloat16*)p.ep_col + n;
        const float ra = p.ep_row_a[m], rb = p.ep_row_b[m];
        if (valid == 32 && ((((uintptr_t)dst) & 15) == 0) && ((((uintptr_t)e) & 15) == 0) &&
            ((((uintptr_t)col) & 15) == 0)) {
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            const uint4 ev = reinterpret_cast<const uint4*>(e)[q];
            const uint4 cv = __ldg(reinterpret_cast<const uint4*>(col) + q);
            const uint32_t ew[4] = {ev.x, ev.y, ev.z, ev.w}, cw[4] = {cv.x, cv.y, cv.z, cv.w};
            uint32_t ow[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
              const float e0 = __uint_as_float(ew[h] << 16), e1 = __uint_as_float(ew[h] & 0xffff0000u);
              const float c0f = __uint_as_float(cw[h] << 16), c1f = __uint_as_float(cw[h] & 0xffff0000u);
              const float a0 = __uint_as_float(v[8 * q + 2 * h]), a1 = __uint_as_float(v[8 * q + 2 * h + 1]);
              ow[h] = pack_bf16x2(ra * c0f * e0 - rb * a0 / c0f, ra * c1f * e1 - rb * a1 / c1f);
            }
            reinterpret_cast<uint4*>(dst)[q] = make_uint4(ow[0], ow[1], ow[2], ow[3]);
          }
        } else {
          for (int q = 0; q < valid; ++q) {
            const float c = __bfloat162float(col[q]);
            dst[q] = __float2bfloat16(ra * c * __bfloat162float(e[q]) - rb * __uint_as_float(v[q]) / c);
          }
        }
      } else if (p.out == OUT_ACT_BWD) {
        // grad_X = grad_Z * f'(reconstructed A): the tile of the reconstructed activation exists only here
        __nv_bfloat16* dst = (__nv_bfloat16*)p.C0 + (int64_t)m * p.ldc + n;
        const __nv_bfloat16* e = (const __nv_bfloat16*)p.ep_E + (int64_t)m * p.ep_ld + n;
        for (int q = 0; q < valid; ++q)
          dst[q] = __float2bfloat16(__bfloat162float(e[q]) * act_derivative(__uint_as_float(v[q]), p.ep_kind));
      } else {
        __nv_bfloat16* dst_hi = (__nv_bfloat16*)p.C0 + (int64_t)m * p.ldc + n;
        __nv_bfloat16* dst_lo = (p.out == OUT_SPLIT && lo_on) ? (__nv_bfloat16*)p.C1 + (int64_t)m * p.ldc + n : nullptr;
        if (valid == 32 && ((((uintptr_t)dst_hi) & 15) == 0)) {
          uint32_t hi[16], lo[16];
#pragma unroll
          for (int q = 0; q < 16; ++q) {
            const float x0 = __uint_as_float(v[2 * q]), x1 = __uint_as_float(v[2 * q + 1]);
            const __nv_bfloat16 h0 = __float2bfloat16(x0), h1 = __float2bfloat16(x1);
            hi[q] = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
            lo[q] = pack_bf16x2(x0 - __bfloat162float(h0), x1 - __bfloat162float(h1));
          }
#pragma unroll
          for (int q = 0; q < 4; ++q)
            reinterpret_cast<uint4*>(dst_hi)[q] = make_uint4(hi[4 * q], hi[4 * q + 1], hi[4 * q + 2], hi[4 * q + 3]);
          if (dst_lo) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
              reinterpret_cast<uint4*>(dst_lo)[q] = make_uint4(lo[4 * q], lo[4 * q + 1], lo[4 * q + 2], lo[4 * q + 3]);
          }
        } else {
          for (int q = 0; q < valid; ++q) {
            const float x = __uint_as_float(v[q]);
            const __nv_bfloat16 h = __float2bfloat16(x);
            dst_hi[q] = h;
            if (dst_lo) dst_lo[q] = __float2bfloat16(x - __bfloat162float(h));
          }
        }
      }
    }
  }
}

// Epilogue of one CTA (eight warps) of the one-tile kernels: waits for the accumulator, then writes it.
// `ring` is the operand ring: once the accumulator is complete every load has landed and every MMA has read
// its stage, so the epilogue warps take the ring over as staging space (8 KB per warp).
__device__ __forceinline__ void tc_epilogue(const TcParams& p, const TmapPack& maps, uint32_t tmem_base,
                                          uint64_t* accum_bar, volatile int* abort_flag_ptr, int warp, int lane,
                                          int m0, int n0, int split, int n_iter, unsigned char* ring) {
  const int m = m0 + (warp & 3) * 32 + lane;
  // OUT_SPLIT with a gate on the low part: read the word while the contraction is still running
  const bool lo_on = !(p.lo_gate != nullptr && *(const volatile uint32_t*)p.lo_gate == 0u);
  bool ok = mbar_wait_bounded(accum_bar, 0, abort_flag_ptr);
  ok = __all_sync(0xffffffffu, ok);
  tc_fence_after();
  if (ok && n_iter > 0) {
    StoreStage st;
    st.base = ring + (uint32_t)(warp - 2) * kStoreWarpBytes;
    st.cnt = 0;
    st.bufs = kStoreBufs;
    tc_store_tile(p, maps, tmem_base, warp, lane, m0, n0, split, st, lo_on);
    stage_drain(st, lane);
  } else if (ok && n_iter == 0 && m < p.M && p.out == OUT_F32 && warp < 6) {
    // an empty K range still owns its partial: write zeros
    float* dst = (float*)p.C0 + (int64_t)split * p.split_stride + (int64_t)m * p.ldc + n0;
    for (int q = 0; q < min(p.bn, p.N - n0); ++q) dst[q] = 0.f;
  }
}

template <bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ TmapPack maps, const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ __align__(8) uint64_t full_bar[kStages];
  __shared__ __align__(8) uint64_t empty_bar[kStages];
  __shared__ __align__(8) uint64_t accum_bar;
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n0 = blockIdx.x * p.bn, m0 = blockIdx.y * kBM, split = blockIdx.z;
  const int kb_begin = split * p.kb_per_split;
  const int kb_count = max(0, min(p.kb_total, kb_begin + p.kb_per_split) - kb_begin);
  int n_iter = kb_count * p.n_terms;
  const uint32_t stage_bytes = kABytes + p.b_bytes;
  // dynamic shared memory is declared 1024-aligned; round up anyway (swizzle atoms need it)
  unsigned char* tiles = (unsigned char*)(((uintptr_t)smem + 1023) & ~(uintptr_t)1023);

  // A gated launch that is not needed leaves before any set-up.  The word may be read this early because it was
  // written at least two kernels back in the stream: this grid only starts once its predecessor has passed its own
  // griddepcontrol.wait, i.e. once everything before the predecessor is complete and visible.  The wait itself is
  // still executed, so that the completion of this grid implies the completion of every earlier one.
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) { pdl_wait(); pdl_launch_dependents(); return; }

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&accum_bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  // everything above overlaps the tail of the previous kernel; global memory only from here on
  pdl_wait();
  pdl_launch_dependents();
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) n_iter = -1;   // every role idles, nothing is stored
  if (p.clear_status && p.dev_status && threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
    *(volatile uint32_t*)p.dev_status = 0u;

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t tx_bytes = stage_bytes;
      for (int it = 0; it < n_iter; ++it) {
        const int s = it % kStages;
        if (!mbar_wait_bounded(&empty_bar[s], ((it / kStages) & 1) ^ 1, &abort_flag)) break;
        const int term = it / kb_count;
        const int k0 = (kb_begin + (it - term * kb_count)) * kBK;
        unsigned char* a_dst = tiles + (size_t)s * stage_bytes;
        unsigned char* b_dst = a_dst + kABytes;
        mbar_arrive_expect_tx(&full_bar[s], tx_bytes);
        if (A_MN) {
          tma_load_2d(a_dst, &maps.a[term], &full_bar[s], m0, k0);
          tma_load_2d(a_dst + 8192, &maps.a[term], &full_bar[s], m0 + 64, k0);
        } else {
          tma_load_2d(a_dst, &maps.a[term], &full_bar[s], k0, m0);
        }
        if (B_MN) {
          for (uint32_t q = 0; q * 8192u < p.b_bytes; ++q)
            tma_load_2d(b_dst + q * 8192u, &maps.b[term], &full_bar[s], n0 + (int)q * 64, k0);
        } else {
          tma_load_2d(b_dst, &maps.b[term], &full_bar[s], k0, n0);
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      // instruction descriptor: fp32 accumulator, bf16 A and B, operand majors, N >> 3, M >> 4
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                             ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(p.bn >> 3) << 17) |
                             ((uint32_t)(kBM >> 4) << 24);
      bool ok = true;
      const int halve_it = p.halve_at_term > 0 ? p.halve_at_term * kb_count : -1;
      for (int it = 0; it < n_iter && ok; ++it) {
        const int s = it % kStages;
        ok = mbar_wait_bounded(&full_bar[s], (it / kStages) & 1, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(tiles + (size_t)s * stage_bytes);
        const uint32_t b_addr = a_addr + kABytes;
        const uint64_t a_desc = make_smem_desc(a_addr, A_MN);
        const uint64_t b_desc = make_smem_desc(b_addr, B_MN);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) {
          // 16 elements along K: 32 bytes inside the swizzled row (K-major) or 16 rows (MN-major)
          const uint64_t a_k = a_desc + (uint64_t)((A_MN ? 2048u : 32u) >> 4) * k;
          const uint64_t b_k = b_desc + (uint64_t)((B_MN ? 2048u : 32u) >> 4) * k;
          if (k == 0 && it == halve_it) tc_mma_bf16_halved(tmem_base, a_k, b_k, idesc);
          else tc_mma_bf16(tmem_base, a_k, b_k, idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit(&empty_bar[s]);  // frees the stage once these MMAs have read it
      }
      tc_commit(&accum_bar);       // accumulator complete (or nothing was issued)
    }
  } else {
    tc_epilogue(p, maps, tmem_base, &accum_bar, &abort_flag, warp, lane, m0, n0, split, n_iter, tiles);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols)
                 : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && p.dev_status) atomicOr(p.dev_status, LORACT_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------------ two CTAs on one tile
// The same contraction with a pair of CTAs (a cluster of two along M) on one 256 x bn tile
// (tcgen05 cta_group::2): each CTA loads its 128 rows of A and HALF of the B tile, the tensor cores of both
// SMs read both halves, and each CTA ends up with its 128 rows of the accumulator in its own tensor
// memory.  Per SM and K block this moves 16 KB + half a B tile instead of 16 KB + a whole one, which is
// what limits the one-CTA kernel when B is re-read from L2 by every CTA; the ring gets six stages.
//   * Both CTAs allocate tensor memory (cta_group::2) and run a TMA producer; the loads of both complete
//     on the full barrier of the even CTA (the leader), which alone issues the MMAs.
//   * tcgen05.commit (cta_group::2, multicast to both CTAs) frees a stage in both CTAs and, at the end,
//     tells both epilogues that the accumulator is complete.
//   * No load uses cluster multicast.
constexpr int kPairStages = 6;

__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
// TMA load whose bytes are counted on a barrier that may live in the peer CTA.
__device__ __forceinline__ void tma_load_2d_pair(void* smem_dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)map), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
// The same load with an L2 eviction-priority hint (a policy made by createpolicy).
__device__ __forceinline__ void tma_load_2d_pair_hint(void* smem_dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                      int x, int y, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint "
      "[%0], [%1, {%3, %4}], [%2], %5;"
      ::"r"(smem_u32(smem_dst)), "l"((uint64_t)map), "r"(bar_cluster_addr), "r"(x), "r"(y), "l"(policy)
      : "memory");
}
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void tc_commit_pair(uint64_t* bar) {
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
      ::"r"(smem_u32(bar)), "h"((uint16_t)3)
      : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                                 uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tc_mma_bf16_pair_halved(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc,
                                                        uint32_t idesc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, 1, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p, 1;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc)
      : "memory");
}

template <bool A_MN, bool B_MN>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_pair_kernel(const __grid_constant__ TmapPack maps, const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ __align__(8) uint64_t full_bar[kPairStages];    // used in the leader: both CTAs' loads of a stage
  __shared__ __align__(8) uint64_t empty_bar[kPairStages];   // in each CTA: the MMAs have read the stage
  __shared__ __align__(8) uint64_t accum_bar;                // in each CTA: the accumulator is complete
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  uint32_t cta_rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(cta_rank));
  const bool leader = cta_rank == 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int half_n = p.bn / 2;                               // B rows (or columns) this CTA loads
  // grid: x = 128-row tiles (the two CTAs of a pair are neighbours in x), y = column tiles, z = K splits.  CTAs start
  // in the order x, then y; the tile a pair works on is taken from that order with the column tile running fastest,
  // so that the pairs that share a row tile of A (pass 1 at r = 512: the same 256 rows of X, two column tiles) run
  // side by side and the second one finds those rows in L2 instead of streaming X from HBM a second time.
  const int pair_lin = (int)(blockIdx.x >> 1) + (int)(gridDim.x >> 1) * (int)blockIdx.y;
  const int tile_m = pair_lin / (int)gridDim.y, tile_n = pair_lin - tile_m * (int)gridDim.y;
  const int n0 = tile_n * p.bn, m0 = (2 * tile_m + (int)cta_rank) * kBM, split = blockIdx.z;
  const int kb_begin = split * p.kb_per_split;
  const int kb_count = max(0, min(p.kb_total, kb_begin + p.kb_per_split) - kb_begin);
  int n_iter = kb_count * p.n_terms;
  const uint32_t stage_bytes = kABytes + p.b_bytes;          // per CTA (b_bytes: half a B tile)
  unsigned char* tiles = (unsigned char*)(((uintptr_t)smem + 1023) & ~(uintptr_t)1023);

  // a gated launch that is not needed: both CTAs of the pair read the same word and leave before any set-up (see the
  // one-CTA kernel for why the word may be read before griddepcontrol.wait)
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) { pdl_wait(); pdl_launch_dependents(); return; }

  if (threadIdx.x == 0) {
    for (int s = 0; s < kPairStages; ++s) { mbar_init(&full_bar[s], 1); mbar_init(&empty_bar[s], 1); }
    mbar_init(&accum_bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  // both CTAs' barriers exist before either CTA signals the other
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  pdl_wait();
  pdl_launch_dependents();
  if (p.gate != nullptr && *(const volatile uint32_t*)p.gate == 0u) n_iter = -1;   // every role idles, nothing is stored
  if (p.clear_status && p.dev_status && threadIdx.x == 0 && blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0)
    *(volatile uint32_t*)p.dev_status = 0u;

  if (warp == 0 || warp == 2) {
    if (lane == 0) {
      const int nb0 = n0 + (int)cta_rank * half_n;           // this CTA's half of the B tile
      // stage, parity, term and K block are carried along (no division in the loop)
      int s = (warp == 0 ? 0 : 1) % kPairStages;
      const uint64_t keep_policy = l2_policy_evict_last();
      uint32_t parity = 1u;
      int term = 0, kb = (warp == 0 ? 0 : 1);
      while (kb >= kb_count && kb_count > 0) { kb -= kb_count; ++term; }
      for (int it = (warp == 0 ? 0 : 1); it < n_iter; it += 2) {
        if (!mbar_wait_bounded(&empty_bar[s], parity, &abort_flag)) break;
        const int k0 = (kb_begin + kb) * kBK;
        const int kb_now = kb;
        unsigned char* a_dst = tiles + (size_t)s * stage_bytes;
        unsigned char* b_dst = a_dst + kABytes;
        // the leader expects the bytes of both CTAs on its barrier
        if (leader) mbar_arrive_expect_tx(&full_bar[s], 2u * stage_bytes);
        const uint32_t bar = map_to_rank(smem_u32(&full_bar[s]), 0u);
        const int term_now = term;
        s += 2; if (s >= kPairStages) { s -= kPairStages; parity ^= 1u; }
        kb += 2; if (kb >= kb_count) { kb -= kb_count; ++term; if (kb >= kb_count) { kb -= kb_count; ++term; } }
        if (A_MN) {
          tma_load_2d_pair(a_dst, &maps.a[term_now], bar, m0, k0);
          tma_load_2d_pair(a_dst + 8192, &maps.a[term_now], bar, m0 + 64, k0);
        } else if (kb_begin + kb_now >= p.a_keep_from_kb) {
          tma_load_2d_pair_hint(a_dst, &maps.a[term_now], bar, k0, m0, keep_policy);
        } else {
          tma_load_2d_pair(a_dst, &maps.a[term_now], bar, k0, m0);
        }
        if (B_MN) {
          for (uint32_t q = 0; q * 8192u < p.b_bytes; ++q)
            tma_load_2d_pair(b_dst + q * 8192u, &maps.b[term_now], bar, nb0 + (int)q * 64, k0);
        } else {
          tma_load_2d_pair(b_dst, &maps.b[term_now], bar, k0, nb0);
        }
      }
    }
    __syncwarp();
  }
  if (warp == 0) {
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // instruction descriptor: fp32 accumulator, bf16 A and B, operand majors, N >> 3, M = 256 >> 4
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((A_MN ? 1u : 0u) << 15) |
                             ((B_MN ? 1u : 0u) << 16) | ((uint32_t)(p.bn >> 3) << 17) |
                             ((uint32_t)((2 * kBM) >> 4) << 24);
      bool ok = true;
      int s = 0;
      uint32_t parity = 0u;
      // descriptors address shared memory in 16-byte units: one addition per stage instead of building them anew
      const uint64_t a_desc0 = make_smem_desc(smem_u32(tiles), A_MN);
      const uint64_t b_desc0 = make_smem_desc(smem_u32(tiles) + kABytes, B_MN);
      const uint32_t stage_units = stage_bytes >> 4;
      const int halve_it = p.halve_at_term > 0 ? p.halve_at_term * kb_count : -1;
      for (int it = 0; it < n_iter && ok; ++it) {
        ok = mbar_wait_bounded(&full_bar[s], parity, &abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint64_t a_desc = a_desc0 + (uint64_t)((uint32_t)s * stage_units);
        const uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)s * stage_units);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) {
          const uint64_t a_k = a_desc + (uint64_t)((A_MN ? 2048u : 32u) >> 4) * k;
          const uint64_t b_k = b_desc + (uint64_t)((B_MN ? 2048u : 32u) >> 4) * k;
          if (k == 0 && it == halve_it) tc_mma_bf16_pair_halved(tmem_base, a_k, b_k, idesc);
          else tc_mma_bf16_pair(tmem_base, a_k, b_k, idesc, (it > 0 || k > 0) ? 1u : 0u);
        }
        tc_commit_pair(&empty_bar[s]);   // frees the stage in both CTAs once these MMAs have read it
        if (++s == kPairStages) { s = 0; parity ^= 1u; }
      }
      tc_commit_pair(&accum_bar);        // accumulator complete in both CTAs (or nothing was issued)
    }
  } else {
    tc_epilogue(p, maps, tmem_base, &accum_bar, &abort_flag, warp, lane, m0, n0, split, n_iter, tiles);
  }
  tc_fence_before();
  __syncthreads();
  // neither CTA frees tensor memory or leaves while the other may still use its shared or tensor memory
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols)
                 : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && p.dev_status) atomicOr(p.dev_status, LORACT_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------------ many tiles per CTA pair, B resident
// C = A B for a short contraction (K <= 512) and a large output, the shape of Reconstruct (X~ = U V): the
// work per output tile is a handful of K blocks, so a kernel that lives for one tile spends its time on set-up,
// one load round trip and one store round trip, none of them overlapped.  Here a CTA pair is persistent:
//   * the tiles are numbered column tile first; pair p takes the contiguous range [p U / P, (p + 1) U / P), so
//     it stays on one column tile for many tiles (and changes it once or twice at most);
//   * its half of the B tile (all K blocks) stays in shared memory while the column tile does not change;
//     only A is streamed through a ring of 128 x 64 stages;
//   * the accumulator is double buffered in tensor memory (2 x bn columns): the tensor cores work on tile
//     i + 1 while the eight epilogue warps read and store tile i.
// Tiles are 256 columns wide whenever the output mode allows it: with 128 columns one instruction keeps the
// tensor pipe busy for 64 cycles, less than the issuing thread needs per instruction (about 100 cycles with
// the fence and the commit of a K block), and the kernel ran issue-bound at about 0.6 of the 256-wide rate.
// Beyond four K blocks the resident B (16 KB per K block and CTA) leaves room for a shorter A ring and one
// staging box per epilogue warp only; the epilogue has the slack (it is about half the tensor time there).
// Barriers.  a_full / a_empty: the ring, as in the pair kernel.  b_full (leader): both halves of B have
// landed; b_empty (each CTA, by commit): every MMA that reads the resident B is done, it may be replaced.
// acc_full[j] (each CTA, by commit): buffer j holds a finished tile; acc_empty[j] (leader, one arrival
// per CTA, sent by the first epilogue warp once all eight have arrived on the CTA's own epi_done[j]): buffer j has been read in both CTAs.  No load uses cluster multicast.
constexpr int kStreamStages = 6;
constexpr int kStreamSmemMax = 226 * 1024;                 // dynamic shared memory the streaming kernel may ask for

// An arrival on a barrier of the peer CTA.  Relaxed: it announces that tensor-memory reads have completed
// (tcgen05.wait::ld has returned), no memory written by this thread has to become visible with it, and a
// releasing arrival at cluster scope costs most of a microsecond.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t bar_cluster_addr) {
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar_cluster_addr) : "memory");
}
__device__ __forceinline__ void mbar_arrive_local(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.b32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster_bounded(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  uint64_t t0 = 0;
  for (uint32_t spin = 1;; ++spin) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((spin & 1023u) == 0u) {
      if (*abort_flag) return false;
      const uint64_t now = global_timer_ns();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitNs) { *abort_flag = 1; return false; }
    }
  }
}

__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_stream_kernel(const __grid_constant__ TmapPack maps, const TcParams p) {
  extern __shared__ __align__(1024) unsigned char smem[];
  __shared__ __align__(8) uint64_t a_full[kStreamStages];
  __shared__ __align__(8) uint64_t a_empty[kStreamStages];
  __shared__ __align__(8) uint64_t b_full, b_empty;
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_empty[2];
  __shared__ __align__(8) uint64_t epi_done[2];
  __shared__ uint32_t tmem_slot;
  __shared__ int abort_flag;

  uint32_t cta_rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(cta_rank));
  const bool leader = cta_rank == 0;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int n_pairs = (int)(gridDim.x >> 1), pair = (int)(blockIdx.x >> 1);
  const int u_begin = (int)((long long)pair * p.st_units / n_pairs);
  const int u_end = (int)((long long)(pair + 1) * p.st_units / n_pairs);
  const int half_n = p.bn / 2;
  const uint32_t b_kb_bytes = p.b_bytes;                     // this CTA's half of B, one K block
  unsigned char* tiles = (unsigned char*)(((uintptr_t)smem + 1023) & ~(uintptr_t)1023);
  unsigned char* b_res = tiles;
  unsigned char* ring = tiles + (size_t)p.kb_total * b_kb_bytes;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStreamStages; ++s) { mbar_init(&a_full[s], 1); mbar_init(&a_empty[s], 1); }
    mbar_init(&b_full, 1);
    mbar_init(&b_empty, 1);
    for (int j = 0; j < 2; ++j) {
      mbar_init(&acc_full[j], 1);
      mbar_init(&acc_empty[j], 2);
      mbar_init(&epi_done[j], kEpiWarps);
    }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  tc_fence_after();
  const uint32_t tmem_base = tmem_slot;
  pdl_wait();
  pdl_launch_dependents();

  if (warp == 0) {
    if (lane == 0) {
      const uint32_t bar_b = map_to_rank(smem_u32(&b_full), 0u);
      int nb = 0, cur_nt = -1;
      int s = 0;                 // ring stage and its phase, carried along (no division in the loop)
      uint32_t ph = 0u;
      bool ok = true;
      for (int u = u_begin; u < u_end && ok; ++u) {
        const int nt = u / p.st_m_tiles, mt = u - nt * p.st_m_tiles;
        if (nt != cur_nt) {
          // the MMAs that read the previous column tile's B are done in both CTAs before it is replaced
          if (nb > 0) ok = mbar_wait_bounded(&b_empty, (uint32_t)((nb - 1) & 1), &abort_flag);
          if (!ok) break;
          if (leader) mbar_arrive_expect_tx(&b_full, 2u * (uint32_t)p.kb_total * b_kb_bytes);
          const int nb0 = nt * p.bn + (int)cta_rank * half_n;
          for (int kb = 0; kb < p.kb_total; ++kb)
            for (uint32_t q = 0; q * 8192u < b_kb_bytes; ++q)
              tma_load_2d_pair(b_res + (size_t)kb * b_kb_bytes + q * 8192u, &maps.b[0], bar_b, nb0 + (int)q * 64,
                               kb * kBK);
          ++nb;
          cur_nt = nt;
        }
        const int m0 = mt * 2 * kBM + (int)cta_rank * kBM;
        for (int kb = 0; kb < p.kb_total; ++kb) {
          ok = mbar_wait_bounded(&a_empty[s], ph ^ 1u, &abort_flag);
          if (!ok) break;
          if (leader) mbar_arrive_expect_tx(&a_full[s], 2u * kABytes);
          tma_load_2d_pair(ring + (size_t)s * kABytes, &maps.a[0], map_to_rank(smem_u32(&a_full[s]), 0u), kb * kBK, m0);
          if (++s == p.st_stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && leader) {
      // instruction descriptor: fp32 accumulator, bf16 A (K-major) and B (MN-major), N >> 3, M = 256 >> 4
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(p.bn >> 3) << 17) |
                             ((uint32_t)((2 * kBM) >> 4) << 24);
      // descriptors address shared memory in 16-byte units: a ring stage is kABytes, a K block of B b_kb_bytes
      const uint64_t a_desc0 = make_smem_desc(smem_u32(ring), false);
      const uint64_t b_desc0 = make_smem_desc(smem_u32(b_res), true);
      int nb = 0, cur_nt = -1;
      int s = 0;                 // ring stage and its phase, carried along (a division here costs 9 % of the kernel)
      uint32_t ph = 0u;
      bool ok = true;
      for (int u = u_begin, ui = 0; u < u_end && ok; ++u, ++ui) {
        const int j = ui & 1;
        const int nt = u / p.st_m_tiles;
        // buffer j was read by both epilogues (the first use of each buffer passes at once)
        ok = mbar_wait_cluster_bounded(&acc_empty[j], (uint32_t)(((ui >> 1) & 1) ^ 1), &abort_flag);
        if (!ok) break;
        if (nt != cur_nt) {
          ok = mbar_wait_bounded(&b_full, (uint32_t)(nb & 1), &abort_flag);
          if (!ok) break;
          ++nb;
          cur_nt = nt;
        }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + (uint32_t)(j * p.bn);
        for (int kb = 0; kb < p.kb_total; ++kb) {
          ok = mbar_wait_bounded(&a_full[s], ph, &abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint64_t a_desc = a_desc0 + (uint64_t)((uint32_t)s * (kABytes >> 4));
          const uint64_t b_desc = b_desc0 + (uint64_t)((uint32_t)kb * (b_kb_bytes >> 4));
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            tc_mma_bf16_pair(d_tmem, a_desc + (uint64_t)(32u >> 4) * k, b_desc + (uint64_t)(2048u >> 4) * k, idesc,
                             (kb > 0 || k > 0) ? 1u : 0u);
          tc_commit_pair(&a_empty[s]);
          if (++s == p.st_stages) { s = 0; ph ^= 1u; }
        }
        if (!ok) break;
        tc_commit_pair(&acc_full[j]);
        if (u + 1 == u_end || (u + 1) / p.st_m_tiles != nt) tc_commit_pair(&b_empty);
      }
    }
  } else {
    bool ok = true;
    StoreStage st;
    st.bufs = (uint32_t)p.store_bufs;
    st.base = ring + (size_t)p.st_stages * kABytes + (uint32_t)(warp - 2) * st.bufs * kStoreBoxBytes;
    st.cnt = 0;
    for (int u = u_begin, ui = 0; u < u_end; ++u, ++ui) {
      const int j = ui & 1;
      const int nt = u / p.st_m_tiles, mt = u - nt * p.st_m_tiles;
      ok = mbar_wait_bounded(&acc_full[j], (uint32_t)((ui >> 1) & 1), &abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
      tc_store_tile(p, maps, tmem_base + (uint32_t)(j * p.bn), warp, lane, mt * 2 * kBM + (int)cta_rank * kBM,
                    nt * p.bn, 0, st);
      // the tile is in registers / shared memory now: hand the buffer back before the stores have drained
      tc_fence_before();
      __syncwarp();
      if (lane == 0) {
        mbar_arrive_local(&epi_done[j]);
        if (warp == 2) {
          // one signal per CTA and tile: the first epilogue warp collects the eight and tells the leader
          if (mbar_wait_bounded(&epi_done[j], (uint32_t)((ui >> 1) & 1), &abort_flag)) {
            if (leader) mbar_arrive_local(&acc_empty[j]);
            else mbar_arrive_cluster(map_to_rank(smem_u32(&acc_empty[j]), 0u));
          }
        }
      }
      __syncwarp();
    }
    stage_drain(st, lane);
  }
  tc_fence_before();
  __syncthreads();
  // neither CTA frees tensor memory or leaves while the other may still use its shared or tensor memory
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols)
                 : "memory");
  }
  if (threadIdx.x == 0 && abort_flag && p.dev_status) atomicOr(p.dev_status, LORACT_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------------ the abort path, exercised on purpose
// One thread waits, with the engine's own bounded wait, on a barrier that nothing ever arrives on.  The wait
// must give up after `limit_ns`, and the kernel then does what every role of the engine does: it records
// LORACT_DEV_WAIT_EXPIRED and returns.  Nothing else runs, so the context stays usable.
__global__ void wait_expiry_probe_kernel(uint32_t* dev_status, uint64_t limit_ns) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool ok = true;
  if (threadIdx.x == 0) ok = mbar_wait_bounded(&bar, 0, &abort_flag, limit_ns);
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag) && dev_status) atomicOr(dev_status, LORACT_DEV_WAIT_EXPIRED);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)sym;
  });
  return fn;
}

// Tensor maps depend only on (pointer, extents, stride, box); they are cached so that a repeated call
// on the same buffers encodes nothing.
typedef std::tuple<const void*, uint64_t, uint64_t, uint64_t, uint32_t, uint32_t, int> TmapKey;
std::mutex g_tmap_mutex;
std::map<TmapKey, CUtensorMap> g_tmap_cache;

// 2-D tensor of bf16 (es = 2) or fp32 (es = 4): `inner` contiguous elements, `outer` rows `ld` elements apart;
// box inner x outer.
cudaError_t get_tmap(const void* ptr, uint64_t inner, uint64_t outer, uint64_t ld, uint32_t box_inner,
                     uint32_t box_outer, CUtensorMap* out, int es = 2) {
  const TmapKey key(ptr, inner, outer, ld, box_inner, box_outer, es);
  {
    std::lock_guard<std::mutex> lock(g_tmap_mutex);
    auto it = g_tmap_cache.find(key);
    if (it != g_tmap_cache.end()) { *out = it->second; return cudaSuccess; }
  }
  EncodeTiledFn fn = get_encode_fn();
  if (!fn) return cudaErrorNotSupported;
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {ld * (uint64_t)es};
  cuuint32_t box[2] = {box_inner, box_outer};
  cuuint32_t elem[2] = {1, 1};
  CUtensorMap m;
  const CUresult r = fn(&m, es == 4 ? CU_TENSOR_MAP_DATA_TYPE_FLOAT32 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box,
                        elem, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B,
                        CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return cudaErrorInvalidValue;
  {
    std::lock_guard<std::mutex> lock(g_tmap_mutex);
    if (g_tmap_cache.size() > 4096) g_tmap_cache.clear();
    g_tmap_cache[key] = m;
  }
  *out = m;
  return cudaSuccess;
}

int pick_bn(int N) {
  const int n16 = (N + 15) / 16 * 16;
  if (n16 <= 256) return n16;
  // widest tile <= 256 that leaves the least padding
  int best = 256, best_pad = ((N + 255) / 256) * 256 - N;
  for (int bn = 256; bn >= 128; bn -= 16) {
    const int pad = ((N + bn - 1) / bn) * bn - N;
    if (pad < best_pad) { best = bn; best_pad = pad; }
  }
  return best;
}

template <bool A_MN, bool B_MN>
cudaError_t launch_variant(const TmapPack& maps, const TcParams& p, dim3 grid, size_t smem, cudaStream_t stream) {
  static std::atomic<bool> configured[64];   // zero-initialised; set once the attribute is in place on a device
  int dev = 0;
  LORACT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    LORACT_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<A_MN, B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kStages * (kABytes + 32768) + 1024));
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  LORACT_CUDA_TRY(launch_pdl(gemm_tc_kernel<A_MN, B_MN>, grid, dim3(kThreads), smem, stream, maps, p));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

template <bool A_MN, bool B_MN>
cudaError_t launch_pair_variant(const TmapPack& maps, const TcParams& p, dim3 grid, size_t smem, cudaStream_t stream) {
  static std::atomic<bool> configured[64];   // zero-initialised; set once the attribute is in place on a device
  int dev = 0;
  LORACT_CUDA_TRY(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64 || !configured[dev].load(std::memory_order_acquire)) {
    LORACT_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_pair_kernel<A_MN, B_MN>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         kPairStages * (kABytes + 16384) + 1024));
    if (dev >= 0 && dev < 64) configured[dev].store(true, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;   // the two CTAs of a pair are neighbours along M
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  LORACT_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_pair_kernel<A_MN, B_MN>, maps, p));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

// Pairs the streaming kernel is launched with: as many as can be resident at once (one CTA per SM).
cudaError_t launch_stream(const TmapPack& maps, TcParams p, size_t smem, cudaStream_t stream) {
  static std::atomic<bool> configured[64];   // zero-initialised; set once the attribute is in place on a device
  static std::atomic<int> max_pairs[64];
  int dev = 0;
  LORACT_CUDA_TRY(cudaGetDevice(&dev));
  const bool cached = dev >= 0 && dev < 64 && configured[dev].load(std::memory_order_acquire);
  int pairs = cached ? max_pairs[dev].load(std::memory_order_relaxed) : 0;
  if (!cached) {
    const int smem_max = kStreamSmemMax;
    LORACT_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_max));
    cudaLaunchConfig_t q = {};
    q.gridDim = dim3(2); q.blockDim = dim3(kThreads); q.dynamicSmemBytes = smem_max;
    cudaLaunchAttribute qa[1];
    qa[0].id = cudaLaunchAttributeClusterDimension;
    qa[0].val.clusterDim.x = 2; qa[0].val.clusterDim.y = 1; qa[0].val.clusterDim.z = 1;
    q.attrs = qa; q.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, gemm_tc_stream_kernel, &q) != cudaSuccess || n < 1) {
      (void)cudaGetLastError();
      cudaDeviceProp prop;
      LORACT_CUDA_TRY(cudaGetDeviceProperties(&prop, dev));
      n = prop.multiProcessorCount / 2;
    }
    pairs = n < 1 ? 1 : n;
    if (dev >= 0 && dev < 64) {
      max_pairs[dev].store(pairs, std::memory_order_relaxed);
      configured[dev].store(true, std::memory_order_release);
    }
  }
  if (pairs > p.st_units) pairs = p.st_units;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * pairs);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  LORACT_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc_stream_kernel, maps, p));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

int g_pair_mode = 1;   // 0: never use the two-CTA kernels (test hook); 1: by shape; 2: as 1, but no streaming kernel

}  // namespace

void gemm_tc_set_pair_mode(int on) { g_pair_mode = on; }

cudaError_t gemm_tc_wait_probe_launch(uint32_t* dev_status, uint64_t limit_ns, cudaStream_t stream) {
  wait_expiry_probe_kernel<<<1, 32, 0, stream>>>(dev_status, limit_ns);
  count_launch(__func__, stream);
  return cudaGetLastError();
}

bool gemm_tc_supported(const GemmDesc& g) {
  if (g.a_type != ELEM_BF16 || g.b_type != ELEM_BF16) return false;
  if (!(g.out == OUT_F32 || g.out == OUT_BF16 || g.out == OUT_SPLIT || g.out == OUT_RMS_BWD || g.out == OUT_ACT_BWD))
    return false;
  if (g.out == OUT_ACT_BWD && (!g.ep_E || g.splits > 1 || g.ep_kind < 0 || g.ep_kind > 1)) return false;
  if (g.out == OUT_RMS_BWD && (!g.ep_E || !g.ep_row_a || !g.ep_row_b || !g.ep_col || g.splits > 1)) return false;
  if (g.M < 1 || g.N < 1 || g.K < 1 || g.n_terms < 1 || g.n_terms > 3) return false;
  if (g.halve_at_term >= g.n_terms) return false;
  if (g.lda % 8 || g.ldb % 8) return false;
  if (g.splits > 1 && g.out != OUT_F32) return false;
  if (g.alpha != 1.0f) return false;
  if (g.accumulate && (g.out != OUT_F32 || g.splits > 1)) return false;
  for (int t = 0; t < g.n_terms; ++t)
    if (((uintptr_t)g.terms[t].A & 15) || ((uintptr_t)g.terms[t].B & 15)) return false;
  return true;
}

int gemm_tc_pick_splits(int M, int N, int K, bool, bool b_mn, int max_splits) {
  const int bn = pick_bn(N);
  const int n_tiles = (N + bn - 1) / bn;
  const int tiles = ((M + kBM - 1) / kBM) * n_tiles;
  const int kb = (K + kBK - 1) / kBK;
  int base = 1;
  if (tiles < 96) {
    base = 148 / tiles;
    if (base > kb / 4) base = kb / 4;  // at least four K blocks per split
    if (base > max_splits) base = max_splits;
    if (base < 1) base = 1;
  }
  // Whole waves: with U units of work on S slots the launch takes ceil(U / S) rounds, so 86 tile pairs on 74 SM
  // pairs cost two full rounds.  Splitting the contraction s ways makes the rounds shorter and fills the last one;
  // it costs the partial sums (s * M * N * 4 bytes, read back by the reduction).  Time in units of one
  // K block (about 0.35 us for a 256 x 256 pair tile); the split count of the simple rule above is kept unless
  // another one is at least 15 % cheaper.
  const bool pair = M >= 2 * kBM && (b_mn ? bn % 128 == 0 : bn % 32 == 0);   // by shape (not by the test hook)
  const long long units = pair ? (long long)((M + 2 * kBM - 1) / (2 * kBM)) * n_tiles : tiles;
  const int slots = pair ? 74 : 148;
  auto cost = [&](int sp) {
    const double rounds = (double)((units * sp + slots - 1) / slots);
    // the partial sums are read back once by the reduction (about 4 TB/s) behind one more launch
    const double reduce_us = sp > 1 ? (double)sp * (double)M * (double)N * 4.0 / 4.0e6 + 4.0 : 0.0;
    return rounds * (double)((kb + sp - 1) / sp) + reduce_us / 0.35;
  };
  int best = base;
  double best_cost = cost(base);
  const int cap = max_splits < 8 ? max_splits : 8;
  for (int sp = 1; sp <= cap; ++sp) {
    if (sp > 1 && kb / sp < 4) break;
    const double c = cost(sp);
    if (c < best_cost && c < 0.85 * cost(base)) { best = sp; best_cost = c; }
  }
  // no empty split: with ceil(kb / best) K blocks each, fewer splits may already cover the contraction (197 blocks
  // in 32 splits of 7 leave three splits with nothing to do but write zeros)
  const int per = (kb + best - 1) / best;
  best = (kb + per - 1) / per;
  return best < 1 ? 1 : best;
}

cudaError_t gemm_tc_launch(const GemmDesc& g, uint32_t* dev_status, cudaStream_t stream) {
  if (!gemm_tc_supported(g)) return cudaErrorNotSupported;
  TcParams p;
  p.M = g.M; p.N = g.N;
  p.bn = pick_bn(g.N);
  p.kb_total = (g.K + kBK - 1) / kBK;
  const int splits = g.splits < 1 ? 1 : g.splits;
  p.kb_per_split = (p.kb_total + splits - 1) / splits;
  p.n_terms = g.n_terms;
  p.out = g.out; p.C0 = g.C0; p.C1 = g.C1; p.ldc = g.ldc; p.split_stride = g.split_stride;
  // Two CTAs per 256-row tile when there are at least 256 rows and the B tile splits into two legal halves.
  const bool pair = g_pair_mode != 0 && g.M >= 2 * kBM && (g.b_mn ? p.bn % 128 == 0 : p.bn % 32 == 0);
  const int b_rows = pair ? p.bn / 2 : p.bn;   // rows (or columns) of B one CTA loads per K block
  p.b_bytes = g.b_mn ? (uint32_t)((b_rows + 63) / 64) * 8192u : (uint32_t)b_rows * 128u;
  p.tmem_cols = 32;
  while ((int)p.tmem_cols < p.bn) p.tmem_cols *= 2;
  p.accumulate = g.accumulate ? 1 : 0;
  p.ep_E = g.ep_E; p.ep_ld = g.ep_ld; p.ep_row_a = g.ep_row_a; p.ep_row_b = g.ep_row_b; p.ep_col = g.ep_col;
  p.ep_kind = g.ep_kind;
  p.dev_status = dev_status;
  p.st_m_tiles = 0; p.st_units = 0; p.tma_store = 0; p.st_stages = kStreamStages; p.store_bufs = kStoreBufs;
  p.halve_at_term = g.halve_at_term > 0 ? g.halve_at_term : 0;
  p.a_keep_from_kb = g.a_keep_from_k >= 0 ? (int)(g.a_keep_from_k / kBK) : p.kb_total;
  p.gate = g.gate;
  p.clear_status = g.clear_status ? 1 : 0;
  p.lo_gate = g.lo_gate;

  TmapPack maps;
  for (int t = 0; t < g.n_terms; ++t) {
    if (g.a_mn) LORACT_CUDA_TRY(get_tmap(g.terms[t].A, g.M, g.K, g.lda, 64, 64, &maps.a[t]));
    else LORACT_CUDA_TRY(get_tmap(g.terms[t].A, g.K, g.M, g.lda, 64, kBM, &maps.a[t]));
    if (g.b_mn) LORACT_CUDA_TRY(get_tmap(g.terms[t].B, g.N, g.K, g.ldb, 64, 64, &maps.b[t]));
    else LORACT_CUDA_TRY(get_tmap(g.terms[t].B, g.K, g.N, g.ldb, 64, (uint32_t)b_rows, &maps.b[t]));
  }
  for (int t = g.n_terms; t < 3; ++t) { maps.a[t] = maps.a[0]; maps.b[t] = maps.b[0]; }
  maps.c[0] = maps.a[0]; maps.c[1] = maps.a[0];
  if (splits == 1) p.split_stride = 0;
  // Output maps for the staged epilogue (boxes of 128 bytes x 32 rows).  Split-K partials are stacked along the
  // rows of one map, which needs them back to back in memory.
  auto staged_ok = [&](int bn) {
    const int es = g.out == OUT_F32 ? 4 : 2;
    if (g.accumulate || bn % (128 / es)) return false;
    if (((uintptr_t)g.C0 & 15) || (g.ldc * es) % 16) return false;
    if (g.out == OUT_SPLIT && ((uintptr_t)g.C1 & 15)) return false;
    if (splits > 1 && g.split_stride != (int64_t)g.M * g.ldc) return false;
    if (g.out == OUT_RMS_BWD && (((uintptr_t)g.ep_E & 15) || ((uintptr_t)g.ep_col & 15) || g.ep_ld % 8)) return false;
    if (g.out == OUT_ACT_BWD && (((uintptr_t)g.ep_E & 15) || g.ep_ld % 8)) return false;
    return true;
  };
  auto make_out_maps = [&]() -> cudaError_t {
    const int es = g.out == OUT_F32 ? 4 : 2;
    const uint32_t box = (uint32_t)(128 / es);
    LORACT_CUDA_TRY(get_tmap(g.C0, g.N, (uint64_t)splits * g.M, g.ldc, box, 32, &maps.c[0], es));
    if (g.out == OUT_SPLIT) LORACT_CUDA_TRY(get_tmap(g.C1, g.N, g.M, g.ldc, box, 32, &maps.c[1], es));
    return cudaSuccess;
  };

  // Short contraction, large output, A K-major, B MN-major, one term (Reconstruct and the pre-norm backward):
  // the persistent kernel with B resident, when there is more than one tile per resident pair.
  if (g_pair_mode == 1 && g.M >= 2 * kBM && !g.a_mn && g.b_mn && g.n_terms == 1 && splits == 1 && p.kb_total <= 8 &&
      g.N >= 256 && g.gate == nullptr && !g.clear_status && g.lo_gate == nullptr) {
    TcParams sp = p;
    // 256 columns per tile (the tensor pipe is issue-bound on narrower instructions).  The resident B takes
    // 16 KB per K block and CTA; beyond four K blocks the A ring and the staging boxes shrink to make room
    // (one box per warp cannot serve the two-box split output, which keeps 128 columns).
    sp.bn = (p.kb_total <= 4 || g.out != OUT_SPLIT) ? 256 : 128;
    sp.b_bytes = (uint32_t)(sp.bn / 2 / 64) * 8192u;
    sp.tmem_cols = 2u * (uint32_t)sp.bn;
    sp.st_stages = kStreamStages;
    sp.store_bufs = kStoreBufs;
    if (sp.bn == 256 && p.kb_total > 4) {
      sp.store_bufs = 1;
      const int room = kStreamSmemMax - 1024 - p.kb_total * (int)sp.b_bytes - kEpiWarps * (int)kStoreBoxBytes;
      sp.st_stages = std::min(kStreamStages, room / (int)kABytes);
    }
    sp.st_m_tiles = (g.M + 2 * kBM - 1) / (2 * kBM);
    const long long units = (long long)sp.st_m_tiles * ((g.N + sp.bn - 1) / sp.bn);
    if (units >= 148 && units < (1ll << 30)) {
      sp.st_units = (int)units;
      sp.tma_store = staged_ok(sp.bn) ? 1 : 0;
      if (sp.tma_store) LORACT_CUDA_TRY(make_out_maps());
      const size_t ssmem = (size_t)sp.kb_total * sp.b_bytes + (size_t)sp.st_stages * kABytes +
                           (size_t)kEpiWarps * sp.store_bufs * kStoreBoxBytes + 1024;
      return launch_stream(maps, sp, ssmem, stream);
    }
  }
  p.tma_store = staged_ok(p.bn) ? 1 : 0;
  if (p.tma_store) LORACT_CUDA_TRY(make_out_maps());
  if (pair) {
    dim3 pgrid(2 * ((g.M + 2 * kBM - 1) / (2 * kBM)), (g.N + p.bn - 1) / p.bn, splits);
    const size_t psmem = (size_t)kPairStages * (kABytes + p.b_bytes) + 1024;
    if (g.a_mn && g.b_mn) return launch_pair_variant<true, true>(maps, p, pgrid, psmem, stream);
    if (g.a_mn && !g.b_mn) return launch_pair_variant<true, false>(maps, p, pgrid, psmem, stream);
    if (!g.a_mn && g.b_mn) return launch_pair_variant<false, true>(maps, p, pgrid, psmem, stream);
    return launch_pair_variant<false, false>(maps, p, pgrid, psmem, stream);
  }
  dim3 grid((g.N + p.bn - 1) / p.bn, (g.M + kBM - 1) / kBM, splits);
  const size_t smem = (size_t)kStages * (kABytes + p.b_bytes) + 1024;
  if (g.a_mn && g.b_mn) return launch_variant<true, true>(maps, p, grid, smem, stream);
  if (g.a_mn && !g.b_mn) return launch_variant<true, false>(maps, p, grid, smem, stream);
  if (!g.a_mn && g.b_mn) return launch_variant<false, true>(maps, p, grid, smem, stream);
  return launch_variant<false, false>(maps, p, grid, smem, stream);
}

}  // namespace loract

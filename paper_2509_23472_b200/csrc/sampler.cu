// Row sampling (the first step of Algorithm 1), the row gather, and the Gaussian test matrix of the RSVD
// comparator.  The generator is Philox4x32-10 (Salmon et al., SC'11), written out here from the
// published round function; it shares no code with the CPU oracle.
#include "common.cuh"

namespace loract {

namespace {

__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

constexpr int kSamplerThreads = 1024;
constexpr int kSamplerMaxRounds = 4096;  // 4M candidates; a permutation of 512 rows needs ~3500
constexpr int kMaxRank = 512;

// One CTA.  Every round draws 1024 candidates in stream order; a candidate survives if no equal value
// stands earlier in the stream (in this round or among those accepted before); survivors are appended
// in stream order until `rank` are found.  This is exactly "the first rank distinct values of the
// stream".  "Stands earlier" is decided with a hash table in shared memory that keeps, for every value
// seen, the smallest stream position it occurred at (atomicMin), so the outcome does not depend on the
// order in which threads run.  The table holds the accepted values (at most 512) and one round of
// candidates (at most 1024), so 2048 slots never fill.
constexpr int kTableSlots = 2048;

__global__ void __launch_bounds__(kSamplerThreads)
sample_indices_kernel(uint32_t seed_lo, uint32_t seed_hi, uint32_t call_lo, uint32_t call_hi,
                      uint32_t n_rows, int rank, int32_t* __restrict__ idx_out,
                      int32_t* __restrict__ idx_copy, uint32_t* __restrict__ dev_status, int clear_status) {
  __shared__ uint32_t accepted[kMaxRank];
  __shared__ uint32_t tab_key[kTableSlots];   // value + 1, 0 = empty
  __shared__ uint32_t tab_pos[kTableSlots];   // smallest stream position of that value
  __shared__ int warp_alive[kSamplerThreads / 32];
  __shared__ int s_count;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  for (int e = tid; e < kTableSlots; e += kSamplerThreads) { tab_key[e] = 0u; tab_pos[e] = 0xFFFFFFFFu; }
  if (tid == 0) s_count = 0;
  __syncthreads();
  for (int round = 0; round < kSamplerMaxRounds; ++round) {
    const int count = s_count;
    if (count >= rank) break;
    const uint32_t i = (uint32_t)round * kSamplerThreads + tid;
    uint32_t w[4];
    philox4x32_10(i >> 2, 0u, call_lo, call_hi, seed_lo, seed_hi, w);
    const uint32_t c = __umulhi(w[i & 3u], n_rows);
    uint32_t h = (c * 2654435761u) >> 21;   // 11 bits
    bool placed = false;
    for (int probe = 0; probe < kTableSlots; ++probe) {
      const uint32_t prev = atomicCAS(&tab_key[h], 0u, c + 1u);
      if (prev == 0u || prev == c + 1u) { placed = true; break; }
      h = (h + 1u) & (kTableSlots - 1);
    }
    if (placed) atomicMin(&tab_pos[h], i);
    __syncthreads();
    const bool alive = placed && tab_pos[h] == i;
    const uint32_t ballot = __ballot_sync(0xffffffffu, alive);
    if (lane == 0) warp_alive[warp] = __popc(ballot);
    __syncthreads();
    int before = 0, total = 0;
    for (int q = 0; q < kSamplerThreads / 32; ++q) {
      const int v = warp_alive[q];
      before += (q < warp) ? v : 0;
      total += v;
    }
    const int pos = count + before + __popc(ballot & ((1u << lane) - 1u));
    if (alive && pos < rank) accepted[pos] = c;
    __syncthreads();
    if (tid == 0) s_count = min(rank, count + total);
    __syncthreads();
  }
  const int found = s_count;
  pdl_wait();   // the index array may still be read by the previous call's kernels
  for (int j = tid; j < rank; j += kSamplerThreads) {
    const int32_t v = (j < found) ? (int32_t)accepted[j] : 0;
    idx_out[j] = v;
    if (idx_copy) idx_copy[j] = v;     // the caller's copy: no separate copy node between this kernel and the gather
  }
  // first kernel of a call: it also clears the status word (no memset node in front of it)
  if (tid == 0 && dev_status) {
    if (clear_status) *dev_status = (found < rank) ? LORACT_DEV_SAMPLER_SHORT : 0u;
    else if (found < rank) atomicOr(dev_status, LORACT_DEV_SAMPLER_SHORT);
  }
}

// dst[row, :] = src[idx[row], :], 16 bytes per thread per step.
__global__ void gather_rows_kernel(const uint4* __restrict__ src, int64_t ld_vec,
                                   const int32_t* __restrict__ idx, int64_t d_vec,
                                   uint4* __restrict__ dst) {
  const int row = blockIdx.y;
  pdl_wait();
  pdl_launch_dependents();
  const int64_t srow = idx[row];
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < d_vec;
       v += (int64_t)gridDim.x * blockDim.x)
    dst[(int64_t)row * d_vec + v] = __ldg(src + srow * ld_vec + v);
}

// The same for one shard of a token-sharded matrix: `src` holds the rows [row0, row0 + n_local) of the whole
// matrix, idx are row numbers of the whole matrix; a sampled row that lives on another shard is written as
// zeros, so that the sum of all shards' results is the gathered matrix.
__global__ void gather_rows_window_kernel(const uint4* __restrict__ src, int64_t ld_vec,
                                          const int32_t* __restrict__ idx, int64_t d_vec, int64_t row0,
                                          int64_t n_local, uint4* __restrict__ dst) {
  const int row = blockIdx.y;
  pdl_wait();
  pdl_launch_dependents();
  const int64_t srow = (int64_t)idx[row] - row0;
  const bool mine = srow >= 0 && srow < n_local;
  for (int64_t v = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; v < d_vec;
       v += (int64_t)gridDim.x * blockDim.x)
    dst[(int64_t)row * d_vec + v] = mine ? __ldg(src + srow * ld_vec + v) : make_uint4(0u, 0u, 0u, 0u);
}

// dst[c][j] = z(j * l + c): element e of the normal stream is z_(e mod 4) of Philox block e div 4,
// u = (w0 + 1) / 2^32, v = w1 / 2^32, z0 = sqrt(-2 ln u) cos(2 pi v), z1 = ... sin(2 pi v).
__global__ void gaussian_rows_kernel(uint32_t seed_lo, uint32_t seed_hi, uint32_t call_lo,
                                     uint32_t call_hi, int l, int64_t d, __nv_bfloat16* __restrict__ dst) {
  const int64_t total = (int64_t)l * d;
  for (int64_t q = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q * 4 < total;
       q += (int64_t)gridDim.x * blockDim.x) {
    uint32_t w[4];
    philox4x32_10((uint32_t)q, 1u, call_lo, call_hi, seed_lo, seed_hi, w);
    float z[4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const float u = ((float)w[2 * h] + 1.0f) * 2.3283064365386963e-10f;
      const float v = (float)w[2 * h + 1] * 2.3283064365386963e-10f;
      const float rad = sqrtf(-2.0f * logf(fminf(u, 1.0f)));
      float s, c;
      sincospif(2.0f * v, &s, &c);
      z[2 * h] = rad * c;
      z[2 * h + 1] = rad * s;
    }
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int64_t e = q * 4 + t;
      if (e < total) {
        const int64_t j = e / l;
        const int c = (int)(e - j * l);
        dst[(int64_t)c * d + j] = __float2bfloat16(z[t]);
      }
    }
  }
}

}  // namespace

cudaError_t sample_indices_launch(uint64_t seed, uint64_t call_id, uint32_t n_rows, int rank,
                                  int32_t* idx_dev, uint32_t* dev_status, cudaStream_t stream, int32_t* idx_copy,
                                  bool clear_status) {
  LORACT_CUDA_TRY(launch_pdl(sample_indices_kernel, dim3(1), dim3(kSamplerThreads), 0, stream, (uint32_t)seed,
                             (uint32_t)(seed >> 32), (uint32_t)call_id, (uint32_t)(call_id >> 32), n_rows, rank,
                             idx_dev, idx_copy, dev_status, clear_status ? 1 : 0));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t gather_rows_launch(const void* src, int64_t ld, const int32_t* idx, int rank, int64_t d,
                               int elem_bytes, void* dst, cudaStream_t stream) {
  const int64_t per_vec = 16 / elem_bytes;
  const int64_t d_vec = d / per_vec, ld_vec = ld / per_vec;
  const int threads = 256;
  int gx = (int)((d_vec + threads - 1) / threads);
  if (gx > 64) gx = 64;
  LORACT_CUDA_TRY(launch_pdl(gather_rows_kernel, dim3(gx, rank), dim3(threads), 0, stream, (const uint4*)src, ld_vec,
                             idx, d_vec, (uint4*)dst));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t gather_rows_window_launch(const void* src, int64_t ld, const int32_t* idx, int rank, int64_t d,
                                      int elem_bytes, int64_t row0, int64_t n_local, void* dst, cudaStream_t stream) {
  const int64_t per_vec = 16 / elem_bytes;
  const int64_t d_vec = d / per_vec, ld_vec = ld / per_vec;
  const int threads = 256;
  int gx = (int)((d_vec + threads - 1) / threads);
  if (gx > 64) gx = 64;
  LORACT_CUDA_TRY(launch_pdl(gather_rows_window_kernel, dim3(gx, rank), dim3(threads), 0, stream, (const uint4*)src,
                             ld_vec, idx, d_vec, row0, n_local, (uint4*)dst));
  count_launch(__func__, stream);
  return cudaGetLastError();
}

cudaError_t gaussian_rows_launch(uint64_t seed, uint64_t call_id, int l, int64_t d,
                                 __nv_bfloat16* dst, cudaStream_t stream) {
  const int64_t blocks4 = ((int64_t)l * d + 3) / 4;
  int grid = (int)((blocks4 + 255) / 256);
  if (grid > 148 * 8) grid = 148 * 8;
  gaussian_rows_kernel<<<grid, 256, 0, stream>>>((uint32_t)seed, (uint32_t)(seed >> 32),
                                                 (uint32_t)call_id, (uint32_t)(call_id >> 32), l, d,
                                                 dst);
  count_launch(__func__, stream);
  return cudaGetLastError();
}

}  // namespace loract

// The C ABI (include/loract.h): argument checks, workspace carving and the sequence of kernel launches
// of each entry point.  All arithmetic happens in the kernels of the other translation units.
#include <atomic>
#include <cstring>
#include <string>
#include <vector>

#include "common.cuh"
#include "../../include/loract_debug.h"

namespace loract {

static std::atomic<uint64_t> g_launches{0};
// ---- stage trace (test hook, one thread at a time): an event behind every launch while it is open
static bool g_trace_open = false;
static std::vector<cudaEvent_t> g_trace_events;
static std::vector<std::string> g_trace_names;
static size_t g_trace_used = 0;
static const char* g_trace_label = "";

static cudaEvent_t trace_event() {
  if (g_trace_used == g_trace_events.size()) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) != cudaSuccess) return nullptr;
    g_trace_events.push_back(e);
  }
  return g_trace_events[g_trace_used++];
}

void trace_label(const char* label) { g_trace_label = label; }

void count_launch(const char* kernel, cudaStream_t stream) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  if (!g_trace_open) return;
  cudaEvent_t e = trace_event();
  if (!e) return;
  cudaEventRecord(e, stream);
  g_trace_names.push_back(std::string(g_trace_label) + " [" + kernel + "]");
}

constexpr int kMaxPowerIters = 8;      // t of Algorithm 1 accepted by loract_compress

loract_status_t check_desc(const loract_desc_t* d) {
  if (!d) return LORACT_ERR_INVALID_ARG;
  if (d->dtype != LORACT_F32 && d->dtype != LORACT_BF16) return LORACT_ERR_INVALID_ARG;
  if (d->reserved != 0) return LORACT_ERR_INVALID_ARG;
  if (d->n_tokens < 1 || d->d < 1 || d->ldx < d->d) return LORACT_ERR_INVALID_ARG;
  if (d->n_tokens > 0x7fffffffLL || d->d > 0x7fffffffLL) return LORACT_ERR_INVALID_ARG;
  if (d->rank < 16 || d->rank > 512 || d->rank % 16) return LORACT_ERR_INVALID_ARG;
  if (d->rank > d->n_tokens || d->rank > d->d) return LORACT_ERR_INVALID_ARG;
  if (d->power_iters < 0) return LORACT_ERR_INVALID_ARG;
  if (d->power_iters > kMaxPowerIters) return LORACT_ERR_UNSUPPORTED;
  const int64_t mult = d->dtype == LORACT_BF16 ? 8 : 4;
  if (d->d % mult || d->ldx % mult) return LORACT_ERR_ALIGNMENT;
  return LORACT_OK;
}
namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

// relative diagonal shifts of the three Cholesky factorisations (fp32 small blocks)
constexpr float kShiftSample = 1e-6f;  // Gram of the sampled rows
// first Gram of the sketch: relative to each diagonal entry itself (W_ii <- W_ii (1 + s)).  The columns of the sketch
// differ in norm by two orders of magnitude and more; a shift relative to the mean diagonal would be of the size of
// the small diagonal entries and leave an orthogonality defect of order one, the entry-relative shift leaves the
// factorisation as accurate as that of the diagonally scaled matrix, whose condition number is a thousand times lower.
constexpr float kShiftFirstDiag = 2e-7f;
constexpr float kShiftFirstMean = 3e-6f;  // fp32 inputs (fp64 factorisation): relative to the mean diagonal
constexpr int kGateWord = 4;               // words 4..6 of the status block: gate, estimate, rounds
constexpr float kShiftSecond = 1e-7f;  // second Gram (already close to the identity), relative to the mean diagonal
// Second orthonormalisation round: run only when est = trace((D W D)^-1) of the first round's Gram matrix
// (D = diag(W)^(-1/2)) times the number of 64-row blocks one accumulation chain of the Gram product covers exceeds
// this, or when a status bit is set.  Measured on B200: the defect max|Q1^T Q1 - I| that one round leaves is about
// 1e-9 * est * blocks (the tensor cores truncate the accumulator once per instruction, so the error of W grows with
// the length of the chain); 2e5 keeps it near 2e-4, under the rounding of U to bf16.
constexpr float kRoundGateDefault = 2.0e5f;
std::atomic<float> g_round_gate{kRoundGateDefault};

struct Carver {
  unsigned char* base;
  size_t off = 0;
  explicit Carver(void* p) : base((unsigned char*)p) {}
  void* take(size_t bytes) {
    void* r = base ? base + off : nullptr;
    off += align_up(bytes);
    return r;
  }
};

inline bool misaligned(const void* p) { return ((uintptr_t)p & 15) != 0; }
inline int elem_bytes(const loract_desc_t* d) { return d->dtype == LORACT_BF16 ? 2 : 4; }

// Workspace of the orthonormalisation + projection of an (n x d) matrix against an l-row test matrix.
struct BasisWs {
  // bf16 path
  __nv_bfloat16 *Lh, *Ll, *Yh, *Yl, *Qh, *Ql;
  float* gram_partials;
  float* v_partials;
  void* sb_scratch;
  // fp32 path
  float *Linv32, *Y32, *Q32, *part32;
  double* gram64;
  int splits_gram_sample, splits_gram, splits_v;
};

struct Plan {
  int64_t n, d;
  int l;
  bool bf16;
  int splits_gs, splits_w, splits_v;
};

inline int simt_splits(int64_t k) {
  int64_t s = k / 128;
  return s < 1 ? 1 : (s > 8 ? 8 : (int)s);
}

Plan make_plan(int64_t n, int64_t d, int l, bool bf16) {
  Plan p;
  p.n = n; p.d = d; p.l = l; p.bf16 = bf16;
  if (bf16) {
    p.splits_gs = gemm_tc_pick_splits(l, l, (int)d, false, false);
    // The tensor cores add every product into the fp32 accumulator with truncation, so a Gram matrix loses about
    // half an ulp per instruction of the chain, with one sign on the diagonal; short chains (up to 64 partial sums,
    // added with rounding afterwards) keep that bias below what one orthonormalisation round tolerates.
    p.splits_w = gemm_tc_pick_splits(l, l, (int)n, true, true, 64);
    p.splits_v = gemm_tc_pick_splits(l, (int)d, (int)n, true, true);
  } else {
    // CUDA-core path: the generic kernel walks K sixteen elements at a time, so a long contraction with few output
    // tiles is split over K (partial sums, added in a fixed order afterwards)
    p.splits_gs = simt_splits(d);
    p.splits_w = simt_splits(n);
    p.splits_v = simt_splits(n);
  }
  return p;
}

void carve_basis(Carver& c, const Plan& p, BasisWs* w) {
  std::memset(w, 0, sizeof(*w));
  const size_t l = (size_t)p.l, n = (size_t)p.n, d = (size_t)p.d;
  w->splits_gram_sample = p.splits_gs; w->splits_gram = p.splits_w; w->splits_v = p.splits_v;
  if (p.bf16) {
    w->Lh = (__nv_bfloat16*)c.take(l * l * 2);
    w->Ll = (__nv_bfloat16*)c.take(l * l * 2);
    // r <= 256 needs none (shared-memory kernel); above that the block scheme keeps W, X and, per level, two
    // (width - 256) x 256 temporaries here
    const size_t lvl1 = l > 256 ? l - 256 : 0, lvl2 = l > 512 ? l - 512 : 0;
    size_t tmp = 2 * 256 * (lvl1 + lvl2);
    if (tmp < 2 * 256 * 256) tmp = 2 * 256 * 256;
    w->sb_scratch = c.take((2 * l * l + tmp) * sizeof(float));
    const size_t gs = (size_t)(p.splits_gs > p.splits_w ? p.splits_gs : p.splits_w);
    w->gram_partials = (float*)c.take(gs * l * l * 4);
    w->Yh = (__nv_bfloat16*)c.take(n * l * 2);
    w->Yl = (__nv_bfloat16*)c.take(n * l * 2);
    w->Qh = (__nv_bfloat16*)c.take(n * l * 2);
    w->Ql = (__nv_bfloat16*)c.take(n * l * 2);
    w->v_partials = (float*)c.take((p.splits_v > 1 ? (size_t)p.splits_v : 0) * l * d * 4);
  } else {
    w->Linv32 = (float*)c.take(l * l * 4);
    w->sb_scratch = c.take((l * l + (l + 31) / 32 * 1024) * sizeof(double));
    const size_t gs = (size_t)(p.splits_gs > p.splits_w ? p.splits_gs : p.splits_w);
    w->gram64 = (double*)c.take(gs * l * l * 8);
    w->Y32 = (float*)c.take(n * l * 4);
    w->Q32 = (float*)c.take(n * l * 4);
    // partial sums of pass 1 (n x l per split over d) and of pass 2 (l x d per split over the tokens)
    const size_t p1 = (size_t)simt_splits((int64_t)d) * n * l, p2 = (size_t)p.splits_v * l * d;
    w->part32 = (float*)c.take((p1 > p2 ? p1 : p2) * 4);
  }
}

cudaError_t run_gemm(const GemmDesc& g, uint32_t* status, cudaStream_t stream) {
  if (gemm_tc_supported(g)) return gemm_tc_launch(g, status, stream);
  return gemm_simt_launch(g, stream);
}

// r x r Gram partials of a K-major matrix S (l x d): S S^T.
cudaError_t gram_rows(const void* S, int l, int64_t d, bool bf16, const BasisWs& w, uint32_t* status,
                      cudaStream_t stream) {
  GemmDesc g;
  g.M = l; g.N = l; g.K = (int)d; g.lda = d; g.ldb = d;
  g.a_type = g.b_type = bf16 ? ELEM_BF16 : ELEM_F32;
  g.terms[0] = {S, S};
  g.ldc = l;
  if (bf16) {
    g.out = OUT_F32; g.C0 = w.gram_partials; g.splits = w.splits_gram_sample;
    g.split_stride = (int64_t)l * l;
  } else {
    g.out = OUT_F64; g.C0 = w.gram64; g.acc64 = true;
    g.splits = w.splits_gram_sample; g.split_stride = (int64_t)l * l;
  }
  return run_gemm(g, status, stream);
}

// fp32 contraction on the CUDA-core kernel, split over K into `splits` partial sums that are then added in a
// fixed order into `out` (M x N, leading dimension N).
cudaError_t simt_split_f32(GemmDesc g, int splits, float* partials, float* out, cudaStream_t stream) {
  if (splits <= 1) { g.out = OUT_F32; g.C0 = out; return gemm_simt_launch(g, stream); }
  g.out = OUT_F32; g.C0 = partials; g.splits = splits; g.split_stride = (int64_t)g.M * g.ldc;
  LORACT_CUDA_TRY(gemm_simt_launch(g, stream));
  return reduce_partials_launch(partials, splits, g.split_stride, g.split_stride, out, nullptr, stream);
}

constexpr double kL2KeepBytes = 48.0 * 1024 * 1024;   // of X, asked to stay in L2 between the two passes (about 20 MB do)
constexpr int kReduceFirst = 8;    // partial count from which a separate, all-SM reduction pays
// `sym`: the partials hold D = Yh^T Yh / 2 + Yh^T Yl (the two-term form of the tall Gram products); the matrix to
// factor is D + D^T.
cudaError_t factor(int l, bool bf16, int n_partials, float shift, const BasisWs& w, uint32_t* status,
                   cudaStream_t stream, bool sym = false, float shift_diag = 0.f, const uint32_t* gate = nullptr,
                   uint32_t* gate_out = nullptr, float gate_threshold = 0.f, bool sum_in_kernel = false) {
  SmallBlockArgs a;
  a.r = l;
  a.shift_diag_rel = shift_diag;
  a.gate = gate;
  a.gate_out = gate_out;
  a.gate_threshold = gate_threshold;
  a.scratch = w.sb_scratch;
  a.dev_status = status;
  if (bf16) {
    a.partials = w.gram_partials; a.partial_type = ELEM_F32; a.n_partials = n_partials;
    a.partial_stride = (int64_t)l * l;
    if (sym) {
      // in place, into the first partial: a CTA of that kernel reads the two tiles it owns from every partial
      // before it writes them, and no other CTA touches them (the scratch area is the factorisation's own)
      LORACT_CUDA_TRY(reduce_sym_launch(w.gram_partials, n_partials, a.partial_stride, l, w.gram_partials, stream, gate));
      a.n_partials = 1;
    } else if (l <= 256 && n_partials >= kReduceFirst && !sum_in_kernel) {
      // The factorisation runs on eight SMs; summing many partials there is a read of several MB through
      // eight SMs' worth of bandwidth.  All SMs sum them first (same order of additions, so the same bits).
      float* W = (float*)w.sb_scratch;
      LORACT_CUDA_TRY(reduce_partials_launch(w.gram_partials, n_partials, a.partial_stride, (int64_t)l * l, W, nullptr,
                                             stream));
      a.partials = W; a.n_partials = 1; a.partial_stride = 0;
    }
    a.use_f64 = false; a.shift_rel = shift;
    a.linv_hi = w.Lh; a.linv_lo = w.Ll;
  } else {
    a.partials = w.gram64; a.partial_type = ELEM_F64; a.n_partials = n_partials; a.partial_stride = (int64_t)l * l;
    a.use_f64 = true; a.shift_rel = shift * 1e-8f;
    a.linv_f32 = w.Linv32;
  }
  return small_block_launch(a, stream);
}

// Omega = L^{-1} T for a test matrix T (l x d, K-major), T T^T = L L^T: the row space of T with rows close to
// orthonormal.  Leaves L^{-1} in w.Lh / w.Ll (w.Linv32).
cudaError_t precondition_rows(const void* T, int l, int64_t d, bool bf16, void* Omega, const BasisWs& w,
                              uint32_t* status, cudaStream_t stream) {
  trace_label("Gram of the test rows");
  LORACT_CUDA_TRY(gram_rows(T, l, d, bf16, w, status, stream));
  trace_label("small block 1");
  LORACT_CUDA_TRY(factor(l, bf16, w.splits_gram_sample, kShiftSample, w, status, stream));
  GemmDesc g;
  g.M = l; g.N = (int)d; g.K = l; g.b_mn = true; g.lda = l; g.ldb = d;
  g.a_type = g.b_type = bf16 ? ELEM_BF16 : ELEM_F32;
  g.ldc = d; g.C0 = Omega;
  if (bf16) {
    g.n_terms = 2; g.terms[0] = {w.Lh, T}; g.terms[1] = {w.Ll, T}; g.out = OUT_BF16;
  } else {
    g.terms[0] = {w.Linv32, T}; g.out = OUT_F32;
  }
  trace_label("Omega = L^-1 T");
  return run_gemm(g, status, stream);
}

// The sketch and the orthonormalisation of Algorithm 1 for a test matrix Omega (l x d, rows are the test vectors):
// Y = X Omega^T, then { W = Y^T Y = L L^T ; Y <- Y L^{-T} }, once or (decided on the device, bf16 inputs) twice.
// U (n x l) receives Q.
cudaError_t range_basis(const void* X, int64_t ldx, const Plan& p, const void* Omega, void* U,
                        const BasisWs& w, uint32_t* status, cudaStream_t stream) {
  const int l = p.l;
  const int n = (int)p.n;
  const int el = p.bf16 ? ELEM_BF16 : ELEM_F32;
  {  // Y = X Omega^T
    GemmDesc g;
    g.M = n; g.N = l; g.K = (int)p.d; g.lda = ldx; g.ldb = p.d; g.a_type = g.b_type = el;
    g.terms[0] = {X, Omega};
    g.ldc = l;
    trace_label("pass 1: Y = X Omega^T");
    if (p.bf16) {
      g.out = OUT_SPLIT; g.C0 = w.Yh; g.C1 = w.Yl;
      // The projection reads X again a few hundred microseconds from now: the last columns this pass streams are
      // asked to stay in L2 (as many bytes of X as kL2KeepBytes).
      const double x_bytes = (double)n * (double)p.d * 2.0;
      if (x_bytes > 0) {
        const double frac = kL2KeepBytes >= x_bytes ? 1.0 : kL2KeepBytes / x_bytes;
        g.a_keep_from_k = (int64_t)((1.0 - frac) * (double)p.d);
      }
      LORACT_CUDA_TRY(run_gemm(g, status, stream));
    } else {
      LORACT_CUDA_TRY(simt_split_f32(g, simt_splits(p.d), w.part32, w.Y32, stream));
    }
  }
  if (!p.bf16) {
    for (int round = 0; round < 2; ++round) {
      const void* Yc = round ? w.Q32 : w.Y32;
      {  // W = Y^T Y
        GemmDesc g;
        g.M = l; g.N = l; g.K = n; g.a_mn = true; g.b_mn = true; g.lda = l; g.ldb = l;
        g.a_type = g.b_type = el;
        g.ldc = l;
        g.terms[0] = {Yc, Yc};
        g.out = OUT_F64; g.C0 = w.gram64; g.acc64 = true;
        g.splits = w.splits_gram; g.split_stride = (int64_t)l * l;
        trace_label(round ? "Gram 2" : "Gram 1");
        LORACT_CUDA_TRY(run_gemm(g, status, stream));
      }
      trace_label(round ? "small block 3" : "small block 2");
      LORACT_CUDA_TRY(factor(l, false, w.splits_gram, round ? kShiftSecond : kShiftFirstMean, w, status, stream, false));
      {  // Y <- Y L^{-T}:  C[m][j] = sum_k Y[m][k] Linv[j][k]
        GemmDesc g;
        g.M = n; g.N = l; g.K = l; g.lda = l; g.ldb = l; g.a_type = g.b_type = el;
        g.ldc = l;
        g.terms[0] = {Yc, w.Linv32};
        g.out = OUT_F32; g.C0 = round == 0 ? (void*)w.Q32 : U;
        trace_label(round ? "apply L^-T 2" : "apply L^-T 1");
        LORACT_CUDA_TRY(run_gemm(g, status, stream));
      }
    }
    return cudaSuccess;
  }
  // bf16 inputs.  Round 1 always runs and writes the leading bf16 part of Q1 = Y L^-T straight into U (the rounded Q1
  // is the result when one round is enough), the remainder into the workspace.  A one-CTA kernel then decides from the
  // factor whether the Gram matrix was conditioned well enough for one round (gate word: 0 = done).  The kernels of
  // round 2 are launched in any case and leave at once when the gate word is zero: no host synchronisation.
  uint32_t* gate_words = status + kGateWord;
  const bool can_gate = l <= 512 && l % 8 == 0;   // widths above 512 (general fp64 kernel) always run both rounds
  const uint32_t* gate = can_gate ? gate_words : nullptr;
  auto gram = [&](const void* Yh, const void* Yl, const uint32_t* gt) {
    // D = (Yl^T Yl + Yh^T Yh) / 2 + Yh^T Yl: the sum of the partials, added to its transpose before the factorisation,
    // is (Yh + Yl)^T (Yh + Yl) with every product kept.  The product of the two low parts is 2^-18 of the diagonal
    // and always positive: left out, it biases every pivot by more than fp32 rounding does.  It goes first, while
    // the accumulator is still small (every instruction truncates the running sum once).
    GemmDesc g;
    g.M = l; g.N = l; g.K = n; g.a_mn = true; g.b_mn = true; g.lda = l; g.ldb = l;
    g.a_type = g.b_type = el;
    g.ldc = l;
    g.n_terms = 3;
    g.terms[0] = {Yl, Yl}; g.terms[1] = {Yh, Yh}; g.terms[2] = {Yh, Yl};
    g.halve_at_term = 2;
    g.out = OUT_F32; g.C0 = w.gram_partials; g.splits = w.splits_gram; g.split_stride = (int64_t)l * l;
    g.gate = gt;
    return run_gemm(g, status, stream);
  };
  auto apply = [&](const void* Yh, const void* Yl, void* Ch, void* Cl, const uint32_t* gt,
                   const uint32_t* lo_gt = nullptr) {
    // C[m][j] = sum_k Y[m][k] Linv[j][k]
    GemmDesc g;
    g.M = n; g.N = l; g.K = l; g.lda = l; g.ldb = l; g.a_type = g.b_type = el;
    g.ldc = l;
    g.n_terms = 3;
    g.terms[0] = {Yh, w.Lh}; g.terms[1] = {Yh, w.Ll}; g.terms[2] = {Yl, w.Lh};
    if (Cl) { g.out = OUT_SPLIT; g.C0 = Ch; g.C1 = Cl; } else { g.out = OUT_BF16; g.C0 = Ch; }
    g.gate = gt;
    g.lo_gate = lo_gt;
    return run_gemm(g, status, stream);
  };
  trace_label("Gram 1");
  LORACT_CUDA_TRY(gram(w.Yh, w.Yl, nullptr));
  const int kb_total = (n + 63) / 64, n_split = w.splits_gram < 1 ? 1 : w.splits_gram;
  const float chain_blocks = (float)((kb_total + n_split - 1) / n_split);
  const float threshold = can_gate ? g_round_gate.load() / chain_blocks : -1.f;
  // up to 256 columns the factorisation kernel forms the estimate itself while it writes L^-1 out
  const bool gate_in_factor = l <= 256 && l % 8 == 0;
  trace_label("small block 2");
  // (widths above 512 take the general fp64 kernel, which knows the shift relative to the mean diagonal only)
  LORACT_CUDA_TRY(factor(l, true, w.splits_gram, l <= 512 ? 0.f : kShiftFirstMean, w, status, stream, true,
                         l <= 512 ? kShiftFirstDiag : 0.f, nullptr, gate_in_factor ? gate_words : nullptr, threshold));
  if (!gate_in_factor) {
    trace_label("round gate");
    LORACT_CUDA_TRY(round_gate_launch(w.gram_partials, w.Lh, l, threshold, status, gate_words, stream));
  }
  trace_label("apply L^-T 1");
  // the remainder of Q1 is only read by the second round: not written when the decision (taken before this kernel
  // starts) is that one round is enough
  LORACT_CUDA_TRY(apply(w.Yh, w.Yl, U, w.Ql, nullptr, gate));
  if (gate_in_factor) {
    // Round 2 is the rare path, and each of its launches costs the common path a few microseconds even when it
    // leaves at once.  So here the Gram matrix is the plain three-term sum (no halving, no symmetrising pass) and the
    // factorisation kernel adds the partial sums itself: three launches instead of four.  Q1 is orthonormal to a few
    // percent, so the product of the two low parts is far below what this round corrects.
    GemmDesc g;
    g.M = l; g.N = l; g.K = n; g.a_mn = true; g.b_mn = true; g.lda = l; g.ldb = l;
    g.a_type = g.b_type = el;
    g.ldc = l;
    g.n_terms = 3;
    g.terms[0] = {U, U}; g.terms[1] = {U, w.Ql}; g.terms[2] = {w.Ql, U};
    g.out = OUT_F32; g.C0 = w.gram_partials; g.splits = w.splits_gram; g.split_stride = (int64_t)l * l;
    g.gate = gate;
    trace_label("Gram 2");
    LORACT_CUDA_TRY(run_gemm(g, status, stream));
    trace_label("small block 3");
    LORACT_CUDA_TRY(factor(l, true, w.splits_gram, kShiftSecond, w, status, stream, false, 0.f, gate, nullptr, 0.f, true));
  } else {
    trace_label("Gram 2");
    LORACT_CUDA_TRY(gram(U, w.Ql, gate));
    trace_label("small block 3");
    LORACT_CUDA_TRY(factor(l, true, w.splits_gram, kShiftSecond, w, status, stream, true, 0.f, gate));
  }
  trace_label("apply L^-T 2");
  // In place when one CTA (pair) owns whole rows of the product: it has read its rows of U and of the remainder
  // completely before its epilogue stores them.  With several column tiles per row block another CTA may still be
  // reading the rows, so the result goes to the workspace and is copied.
  GemmDesc probe;
  probe.M = n; probe.N = l; probe.K = l; probe.lda = l; probe.ldb = l; probe.ldc = l; probe.n_terms = 3;
  probe.terms[0] = {U, w.Lh}; probe.terms[1] = {U, w.Ll}; probe.terms[2] = {w.Ql, w.Lh};
  probe.out = OUT_BF16; probe.C0 = U;
  if (l <= 256 && gemm_tc_supported(probe)) {
    LORACT_CUDA_TRY(apply(U, w.Ql, U, nullptr, gate));
  } else {
    LORACT_CUDA_TRY(apply(U, w.Ql, w.Qh, nullptr, gate));
    if (gate) {
      LORACT_CUDA_TRY(copy_bf16_gated_launch(w.Qh, (__nv_bfloat16*)U, (int64_t)n * l, gate, stream));
    } else {
      LORACT_CUDA_TRY(cudaMemcpyAsync(U, w.Qh, (size_t)n * l * 2, cudaMemcpyDeviceToDevice, stream));
    }
  }
  return cudaSuccess;
}

// The projection step of Algorithm 1: V = U^T X  (l x d), from the stored U.
cudaError_t project(const void* U, const void* X, int64_t ldx, const Plan& p, void* V, const BasisWs& w,
                    uint32_t* status, cudaStream_t stream) {
  GemmDesc g;
  g.M = p.l; g.N = (int)p.d; g.K = (int)p.n; g.a_mn = true; g.b_mn = true; g.lda = p.l; g.ldb = ldx;
  g.a_type = g.b_type = p.bf16 ? ELEM_BF16 : ELEM_F32;
  g.terms[0] = {U, X};
  g.ldc = p.d;
  trace_label("pass 2: V = U^T X");
  if (!p.bf16) return simt_split_f32(g, w.splits_v, w.part32, (float*)V, stream);
  if (w.splits_v <= 1) { g.out = OUT_BF16; g.C0 = V; return run_gemm(g, status, stream); }
  g.out = OUT_F32; g.C0 = w.v_partials; g.splits = w.splits_v; g.split_stride = (int64_t)p.l * p.d;
  LORACT_CUDA_TRY(run_gemm(g, status, stream));
  return reduce_partials_launch(w.v_partials, w.splits_v, g.split_stride, g.split_stride, nullptr,
                                (__nv_bfloat16*)V, stream);
}

// ------------------------------------------------------------------ compress
struct CompressWs {
  uint32_t* status;
  int32_t* idx;
  void* S;      // sampled rows, l x d
  void* Omega;  // preconditioned test matrix, l x d
  void* A;      // normalised input of the pre-norm entry (only when it is not returned)
  BasisWs b;
};

size_t carve_compress(void* ws, const loract_desc_t* desc, bool with_A, CompressWs* out, Plan* plan) {
  const bool bf16 = desc->dtype == LORACT_BF16;
  *plan = make_plan(desc->n_tokens, desc->d, desc->rank, bf16);
  Carver c(ws);
  CompressWs w;
  w.status = (uint32_t*)c.take(256);
  w.idx = (int32_t*)c.take((size_t)desc->rank * 4);
  const size_t es = (size_t)elem_bytes(desc);
  w.S = c.take((size_t)desc->rank * desc->d * es);
  w.Omega = c.take((size_t)desc->rank * desc->d * es);
  carve_basis(c, *plan, &w.b);
  w.A = with_A ? c.take((size_t)desc->n_tokens * desc->d * es) : nullptr;
  if (out) *out = w;
  return c.off;
}

// Algorithm 1, t = 0, on a matrix X that is already in place.
cudaError_t compress_core(const loract_desc_t* desc, const void* X, int64_t ldx, void* U, void* V,
                          int32_t* idx_out, const CompressWs& w, const Plan& plan, cudaStream_t stream) {
  const bool bf16 = plan.bf16;
  const int r = desc->rank;
  // the sampling step: sample rows, gather them.  The sampler is the first kernel of the call: it clears the status word
  // and writes the caller's copy of the indices itself.
  trace_label("sample");
  LORACT_CUDA_TRY(sample_indices_launch(desc->seed, desc->call_id, (uint32_t)desc->n_tokens, r, w.idx,
                                        w.status, stream, idx_out, true));
  trace_label("gather");
  LORACT_CUDA_TRY(gather_rows_launch(X, ldx, w.idx, r, desc->d, elem_bytes(desc), w.S, stream));
  // From the sketch to the orthonormal basis.  The test matrix (the sampled rows A_k at first, Q^T X in the power
  // iterations of the loop
  // 3 to 6) is preconditioned before every product with X: with T T^T = L L^T, Omega = L^{-1} T has the row
  // space of T, so range(X Omega^T) = range(X T^T), but its rows are close to orthonormal, which keeps the
  // spectrum of the sketch from being squared (and, in the iterations, raised to the fourth power).
  for (int it = 0; it <= desc->power_iters; ++it) {
    LORACT_CUDA_TRY(precondition_rows(w.S, r, desc->d, bf16, w.Omega, w.b, w.status, stream));
    // Y = X Omega^T, Y = QR (Q written to U)
    LORACT_CUDA_TRY(range_basis(X, ldx, plan, w.Omega, U, w.b, w.status, stream));
    // inside the power-iteration loop: the next test matrix is (X^T Q)^T = Q^T X, kept where A_k was
    if (it < desc->power_iters) LORACT_CUDA_TRY(project(U, X, ldx, plan, w.S, w.b, w.status, stream));
  }
  // the projection: V = U^T X
  return project(U, X, ldx, plan, V, w.b, w.status, stream);
}

struct WgradWs {
  float* partials;
  float* T;                      // fp32 path
  __nv_bfloat16 *Th, *Tm, *Tl;   // bf16 path: T as a bf16 triple, leading dimension g rounded up to 8
  int splits;
  int g8;
};
size_t carve_wgrad(void* ws, const loract_desc_t* desc, int g, WgradWs* out) {
  Carver c(ws);
  c.take(256);
  WgradWs w;
  w.splits = desc->dtype == LORACT_BF16 ? gemm_tc_pick_splits(desc->rank, g, (int)desc->n_tokens, true, true)
                                        : 2 * simt_splits(desc->n_tokens);
  w.partials = (float*)c.take((size_t)w.splits * desc->rank * g * 4);
  w.T = (float*)c.take((size_t)desc->rank * g * 4);
  w.g8 = (g + 7) / 8 * 8;
  w.Th = (__nv_bfloat16*)c.take((size_t)desc->rank * w.g8 * 2);
  w.Tm = (__nv_bfloat16*)c.take((size_t)desc->rank * w.g8 * 2);
  w.Tl = (__nv_bfloat16*)c.take((size_t)desc->rank * w.g8 * 2);
  if (out) *out = w;
  return c.off;
}

// ------------------------------------------------------------------ joint compression of a token-sharded X
// Every shard runs the same stages on its rows; between stages the caller adds the small matrices the stages
// hand out over all shards (the sampled rows, the r x r Gram matrices, V).  State between stages (the test matrix,
// the sketch, the once-orthonormalised sketch, L^-1) stays in the shard's workspace.
struct JointWs {
  uint32_t* status;
  int32_t* idx;
  void* Omega;
  BasisWs b;
};

size_t carve_joint(void* ws, const loract_desc_t* desc, JointWs* out, Plan* plan) {
  *plan = make_plan(desc->n_tokens, desc->d, desc->rank, true);
  Carver c(ws);
  JointWs w;
  w.status = (uint32_t*)c.take(256);
  w.idx = (int32_t*)c.take((size_t)desc->rank * 4);
  w.Omega = c.take((size_t)desc->rank * desc->d * 2);
  carve_basis(c, *plan, &w.b);
  if (out) *out = w;
  return c.off;
}

// W (l x l fp32, summed over this shard's split-K partials) = Y^T Y for a tall bf16 pair Y = Yh + Yl (n x l).
cudaError_t gram_tall_sum(const void* Yh, const void* Yl, int n, int l, const BasisWs& w, float* W, uint32_t* status,
                          cudaStream_t stream) {
  GemmDesc g;
  g.M = l; g.N = l; g.K = n; g.a_mn = true; g.b_mn = true; g.lda = l; g.ldb = l;
  // two terms, the first halved: the partials sum to D with D + D^T = Yh^T Yh + Yh^T Yl + Yl^T Yh
  g.n_terms = 2;
  g.terms[0] = {Yh, Yh}; g.terms[1] = {Yh, Yl};
  g.halve_at_term = 1;
  g.out = OUT_F32; g.ldc = l;
  const int splits = w.splits_gram < 1 ? 1 : w.splits_gram;
  g.C0 = w.gram_partials; g.splits = splits; g.split_stride = (int64_t)l * l;
  LORACT_CUDA_TRY(run_gemm(g, status, stream));
  return reduce_sym_launch(w.gram_partials, splits, g.split_stride, l, W, stream);
}

// L^-1 (bf16 pair in w.Lh / w.Ll) from one summed l x l Gram matrix.
cudaError_t factor_matrix(const float* W, int l, float shift, const BasisWs& w, uint32_t* status, cudaStream_t stream) {
  SmallBlockArgs a;
  a.r = l; a.scratch = w.sb_scratch; a.dev_status = status;
  a.partials = W; a.partial_type = ELEM_F32; a.n_partials = 1; a.partial_stride = (int64_t)l * l;
  a.use_f64 = false; a.shift_rel = shift;
  a.linv_hi = w.Lh; a.linv_lo = w.Ll;
  return small_block_launch(a, stream);
}

// C = Y L^-T for a tall bf16 pair Y (n x l): as a bf16 pair (Ch, Cl) or, with Cl == nullptr, rounded once to bf16.
cudaError_t apply_linv(const void* Yh, const void* Yl, int n, int l, const BasisWs& w, void* Ch, void* Cl,
                       uint32_t* status, cudaStream_t stream) {
  GemmDesc g;
  g.M = n; g.N = l; g.K = l; g.lda = l; g.ldb = l; g.ldc = l;
  g.n_terms = 3;
  g.terms[0] = {Yh, w.Lh}; g.terms[1] = {Yh, w.Ll}; g.terms[2] = {Yl, w.Lh};
  if (Cl) { g.out = OUT_SPLIT; g.C0 = Ch; g.C1 = Cl; } else { g.out = OUT_BF16; g.C0 = Ch; }
  return run_gemm(g, status, stream);
}

loract_status_t check_joint(const loract_desc_t* desc) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (desc->dtype != LORACT_BF16 || desc->power_iters != 0) return LORACT_ERR_UNSUPPORTED;
  return LORACT_OK;
}

std::atomic<int> g_last_cuda_error{0};
loract_status_t from_cuda(cudaError_t e) {
  if (e == cudaSuccess) return LORACT_OK;
  g_last_cuda_error.store((int)e, std::memory_order_relaxed);
  return LORACT_ERR_CUDA;
}

}  // namespace
}  // namespace loract

using namespace loract;

extern "C" {

size_t loract_workspace_bytes(const loract_desc_t* desc) {
  if (check_desc(desc) != LORACT_OK) return 0;
  Plan plan;
  size_t a = carve_compress(nullptr, desc, /*with_A=*/true, nullptr, &plan);
  size_t b = carve_wgrad(nullptr, desc, 256, nullptr);
  return a > b ? a : b;
}

loract_status_t loract_sample_indices(const loract_desc_t* desc, int32_t* idx_dev, void* ws, size_t ws_bytes,
                                      void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (!idx_dev || !ws) return LORACT_ERR_INVALID_ARG;
  if (ws_bytes < 256) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(ws, 0, 4, st);
  if (e == cudaSuccess)
    e = sample_indices_launch(desc->seed, desc->call_id, (uint32_t)desc->n_tokens, desc->rank, idx_dev,
                              (uint32_t*)ws, st);
  return from_cuda(e);
}

loract_status_t loract_compress(const loract_desc_t* desc, const void* X, void* U, void* V, int32_t* idx_out,
                                void* ws, size_t ws_bytes, void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (!X || !U || !V || !ws) return LORACT_ERR_INVALID_ARG;
  if (misaligned(X) || misaligned(U) || misaligned(V) || ((uintptr_t)ws & 255)) return LORACT_ERR_ALIGNMENT;
  CompressWs w;
  Plan plan;
  const size_t need = carve_compress(ws, desc, /*with_A=*/false, &w, &plan);
  if (ws_bytes < need) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  return from_cuda(compress_core(desc, X, desc->ldx, U, V, idx_out, w, plan, (cudaStream_t)stream));
}

loract_status_t loract_compress_prenorm(const loract_desc_t* desc, const void* X, const void* gamma,
                                        const void* beta, float eps, int32_t kind, void* A_out, float* rstd,
                                        float* mean, void* U, void* V, int32_t* idx_out, void* ws,
                                        size_t ws_bytes, void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (!X || !gamma || !rstd || !U || !V || !ws) return LORACT_ERR_INVALID_ARG;
  if (kind != LORACT_NORM_RMS && kind != LORACT_NORM_LAYER) return LORACT_ERR_INVALID_ARG;
  if (kind == LORACT_NORM_LAYER && !mean) return LORACT_ERR_INVALID_ARG;
  if (!(eps >= 0.f)) return LORACT_ERR_INVALID_ARG;
  if (misaligned(X) || misaligned(U) || misaligned(V) || (A_out && misaligned(A_out)) || ((uintptr_t)ws & 255))
    return LORACT_ERR_ALIGNMENT;
  CompressWs w;
  Plan plan;
  const size_t need = carve_compress(ws, desc, /*with_A=*/A_out == nullptr, &w, &plan);
  if (ws_bytes < need) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  void* A = A_out ? A_out : w.A;
  cudaError_t e = norm_forward_launch(X, desc->n_tokens, desc->d, desc->ldx,
                                      desc->dtype == LORACT_BF16 ? ELEM_BF16 : ELEM_F32, gamma, beta, eps, kind,
                                      A, desc->d, rstd, kind == LORACT_NORM_LAYER ? mean : nullptr, st);
  if (e != cudaSuccess) return LORACT_ERR_CUDA;
  return from_cuda(compress_core(desc, A, desc->d, U, V, idx_out, w, plan, st));
}

loract_status_t loract_reconstruct(const loract_desc_t* desc, const void* U, const void* V, void* X_out,
                                   void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (!U || !V || !X_out) return LORACT_ERR_INVALID_ARG;
  if (misaligned(U) || misaligned(V) || misaligned(X_out)) return LORACT_ERR_ALIGNMENT;
  const bool bf16 = desc->dtype == LORACT_BF16;
  GemmDesc g;
  g.M = (int)desc->n_tokens; g.N = (int)desc->d; g.K = desc->rank; g.b_mn = true;
  g.lda = desc->rank; g.ldb = desc->d;
  g.a_type = g.b_type = bf16 ? ELEM_BF16 : ELEM_F32;
  g.terms[0] = {U, V};
  g.out = bf16 ? OUT_BF16 : OUT_F32; g.C0 = X_out; g.ldc = desc->ldx;
  return from_cuda(run_gemm(g, nullptr, (cudaStream_t)stream));
}

loract_status_t loract_weight_grad(const loract_desc_t* desc, const void* U, const void* V, const void* G,
                                   int32_t g, int64_t ldg, float* dW, int accumulate, void* ws, size_t ws_bytes,
                                   void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (!U || !V || !G || !dW || !ws) return LORACT_ERR_INVALID_ARG;
  if (g < 1 || g > 256 || ldg < g) return LORACT_ERR_INVALID_ARG;
  if (misaligned(U) || misaligned(V) || misaligned(G) || ((uintptr_t)ws & 255)) return LORACT_ERR_ALIGNMENT;
  if (ldg % (desc->dtype == LORACT_BF16 ? 8 : 4)) return LORACT_ERR_ALIGNMENT;
  WgradWs w;
  const size_t need = carve_wgrad(ws, desc, g, &w);
  if (ws_bytes < need) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const int el = desc->dtype == LORACT_BF16 ? ELEM_BF16 : ELEM_F32;
  const int r = desc->rank;
  GemmDesc t;  // T = U^T G  (r x g), split over tokens
  t.M = r; t.N = g; t.K = (int)desc->n_tokens; t.a_mn = true; t.b_mn = true; t.lda = r; t.ldb = ldg;
  t.a_type = t.b_type = el;
  t.terms[0] = {U, G};
  t.out = OUT_F32; t.C0 = w.partials; t.ldc = g; t.splits = w.splits; t.split_stride = (int64_t)r * g;
  uint32_t* status = (uint32_t*)ws;
  trace_label("weight grad");
  // the first kernel clears the status word itself where it can (tensor-core path); a memset node otherwise
  cudaError_t e = cudaSuccess;
  if (gemm_tc_supported(t)) t.clear_status = true;
  else e = cudaMemsetAsync(status, 0, 4, st);
  if (e == cudaSuccess) e = run_gemm(t, status, st);
  if (e == cudaSuccess && el == ELEM_BF16) {
    // dW = V^T T on the tensor cores: T (fp32) is carried as a bf16 triple, so that the three products
    // together are as accurate as one fp32 product
    e = reduce_split3_launch(w.partials, w.splits, t.split_stride, r, g, g, w.g8, w.Th, w.Tm, w.Tl, st);
    GemmDesc q;
    q.M = (int)desc->d; q.N = g; q.K = r; q.a_mn = true; q.b_mn = true; q.lda = desc->d; q.ldb = w.g8;
    q.n_terms = 3;
    q.terms[0] = {V, w.Th}; q.terms[1] = {V, w.Tm}; q.terms[2] = {V, w.Tl};
    q.out = OUT_F32; q.C0 = dW; q.ldc = g; q.accumulate = accumulate != 0;
    if (e == cudaSuccess && gemm_tc_supported(q)) return from_cuda(gemm_tc_launch(q, status, st));
  }
  if (e == cudaSuccess)
    e = reduce_partials_launch(w.partials, w.splits, t.split_stride, t.split_stride, w.T, nullptr, st);
  if (e == cudaSuccess) {
    GemmDesc q;  // dW = V^T T  (d x g)
    q.M = (int)desc->d; q.N = g; q.K = r; q.a_mn = true; q.b_mn = true; q.lda = desc->d; q.ldb = g;
    q.a_type = el; q.b_type = ELEM_F32;
    q.terms[0] = {V, w.T};
    q.out = OUT_F32; q.C0 = dW; q.ldc = g; q.accumulate = accumulate != 0;
    e = gemm_simt_launch(q, st);
  }
  return from_cuda(e);
}

size_t loract_prenorm_backward_workspace_bytes(const loract_desc_t* desc) {
  if (check_desc(desc) != LORACT_OK) return 0;
  Carver c(nullptr);
  c.take(256);
  c.take((size_t)desc->n_tokens * desc->rank * 4);   // P = grad_A V^T
  c.take((size_t)desc->n_tokens * 4);                // row_a
  c.take((size_t)desc->n_tokens * 4);                // row_b
  return c.off;
}

loract_status_t loract_prenorm_backward(const loract_desc_t* desc, const void* U, const void* V, const void* gamma,
                                        const float* rstd, const void* grad_A, void* grad_X, void* ws,
                                        size_t ws_bytes, void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (desc->dtype != LORACT_BF16) return LORACT_ERR_UNSUPPORTED;
  if (!U || !V || !gamma || !rstd || !grad_A || !grad_X || !ws) return LORACT_ERR_INVALID_ARG;
  if (misaligned(U) || misaligned(V) || misaligned(gamma) || misaligned(grad_A) || misaligned(grad_X) ||
      ((uintptr_t)ws & 255))
    return LORACT_ERR_ALIGNMENT;
  if (ws_bytes < loract_prenorm_backward_workspace_bytes(desc)) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  const int n = (int)desc->n_tokens, d = (int)desc->d, r = desc->rank;
  Carver c(ws);
  uint32_t* status = (uint32_t*)c.take(256);
  float* P = (float*)c.take((size_t)n * r * 4);
  float* row_a = (float*)c.take((size_t)n * 4);
  float* row_b = (float*)c.take((size_t)n * 4);
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(status, 0, 4, st);
  // With A~ = U V: (grad_Xbar . Xbar)_ij = grad_A_ij A~_ij (gamma cancels), so the row mean of Section 3.3 is
  // (1 / d) U_i . (grad_A V^T)_i -- a tall-skinny product instead of a pass over a reconstructed matrix.
  if (e == cudaSuccess) {
    GemmDesc g;
    g.M = n; g.N = r; g.K = d; g.lda = desc->ldx; g.ldb = d;
    g.terms[0] = {grad_A, V};
    g.out = OUT_F32; g.C0 = P; g.ldc = r;
    trace_label("pre-norm backward: P = grad_A V^T");
    e = gemm_tc_supported(g) ? gemm_tc_launch(g, status, st) : cudaErrorNotSupported;
  }
  if (e == cudaSuccess) {
    trace_label("pre-norm backward: row coefficients");
    e = rms_backward_rows_launch((const __nv_bfloat16*)U, P, rstd, n, r, d, row_a, row_b, st);
  }
  if (e == cudaSuccess) {
    // grad_X = rstd * (grad_A * gamma - (A~ / gamma) * inner), A~ tile by tile in tensor memory only
    GemmDesc g;
    g.M = n; g.N = d; g.K = r; g.b_mn = true; g.lda = r; g.ldb = d;
    g.terms[0] = {U, V};
    g.out = OUT_RMS_BWD; g.C0 = grad_X; g.ldc = desc->ldx;
    g.ep_E = grad_A; g.ep_ld = desc->ldx; g.ep_row_a = row_a; g.ep_row_b = row_b; g.ep_col = gamma;
    trace_label("pre-norm backward: grad_X");
    e = gemm_tc_supported(g) ? gemm_tc_launch(g, status, st) : cudaErrorNotSupported;
  }
  return from_cuda(e);
}

loract_status_t loract_activation_backward(const loract_desc_t* desc, const void* U, const void* V,
                                           const void* grad_Z, int32_t kind, void* grad_X, void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (desc->dtype != LORACT_BF16) return LORACT_ERR_UNSUPPORTED;
  if (kind != LORACT_ACT_SILU && kind != LORACT_ACT_GELU) return LORACT_ERR_INVALID_ARG;
  if (!U || !V || !grad_Z || !grad_X) return LORACT_ERR_INVALID_ARG;
  if (misaligned(U) || misaligned(V) || misaligned(grad_Z) || misaligned(grad_X)) return LORACT_ERR_ALIGNMENT;
  // grad_X = grad_Z * f'(A~), A~ = U V tile by tile in tensor memory only: the epilogue of the reconstruct
  // contraction takes the derivative and multiplies
  GemmDesc g;
  g.M = (int)desc->n_tokens; g.N = (int)desc->d; g.K = desc->rank; g.b_mn = true;
  g.lda = desc->rank; g.ldb = desc->d;
  g.terms[0] = {U, V};
  g.out = OUT_ACT_BWD; g.C0 = grad_X; g.ldc = desc->ldx;
  g.ep_E = grad_Z; g.ep_ld = desc->ldx; g.ep_kind = kind;
  trace_label("activation backward: grad_X");
  if (!gemm_tc_supported(g)) return LORACT_ERR_UNSUPPORTED;
  return from_cuda(gemm_tc_launch(g, nullptr, (cudaStream_t)stream));
}

size_t loract_joint_workspace_bytes(const loract_desc_t* desc) {
  if (check_joint(desc) != LORACT_OK) return 0;
  Plan plan;
  return carve_joint(nullptr, desc, nullptr, &plan);
}

loract_status_t loract_joint_sample_rows(const loract_desc_t* desc, int64_t n_global, int64_t row0, const void* X_local,
                                         void* S, int32_t* idx_out, void* ws, size_t ws_bytes, void* stream) {
  loract_status_t s = check_joint(desc);
  if (s != LORACT_OK) return s;
  if (!X_local || !S || !ws) return LORACT_ERR_INVALID_ARG;
  if (n_global < desc->n_tokens || n_global > 0x7fffffffLL || row0 < 0 || row0 + desc->n_tokens > n_global ||
      desc->rank > n_global)
    return LORACT_ERR_INVALID_ARG;
  if (misaligned(X_local) || misaligned(S) || ((uintptr_t)ws & 255)) return LORACT_ERR_ALIGNMENT;
  JointWs w;
  Plan plan;
  if (ws_bytes < carve_joint(ws, desc, &w, &plan)) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  trace_label("joint: sample");
  cudaError_t e = sample_indices_launch(desc->seed, desc->call_id, (uint32_t)n_global, desc->rank, w.idx, w.status, st,
                                        idx_out, true);
  trace_label("joint: gather own rows");
  if (e == cudaSuccess)
    e = gather_rows_window_launch(X_local, desc->ldx, w.idx, desc->rank, desc->d, 2, row0, desc->n_tokens, S, st);
  return from_cuda(e);
}

loract_status_t loract_joint_sketch(const loract_desc_t* desc, const void* X_local, const void* S_sum, float* W_partial,
                                    void* ws, size_t ws_bytes, void* stream) {
  loract_status_t s = check_joint(desc);
  if (s != LORACT_OK) return s;
  if (!X_local || !S_sum || !W_partial || !ws) return LORACT_ERR_INVALID_ARG;
  if (misaligned(X_local) || misaligned(S_sum) || misaligned(W_partial) || ((uintptr_t)ws & 255))
    return LORACT_ERR_ALIGNMENT;
  JointWs w;
  Plan plan;
  if (ws_bytes < carve_joint(ws, desc, &w, &plan)) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const int r = desc->rank, n = (int)desc->n_tokens;
  // the test matrix from the complete sampled rows: the same bits on every shard
  cudaError_t e = precondition_rows(S_sum, r, desc->d, true, w.Omega, w.b, w.status, st);
  if (e == cudaSuccess) {  // this shard's rows of the sketch, Y = X_local Omega^T
    GemmDesc g;
    g.M = n; g.N = r; g.K = (int)desc->d; g.lda = desc->ldx; g.ldb = desc->d;
    g.terms[0] = {X_local, w.Omega};
    g.ldc = r; g.out = OUT_SPLIT; g.C0 = w.b.Yh; g.C1 = w.b.Yl;
    trace_label("joint: pass 1");
    e = run_gemm(g, w.status, st);
  }
  trace_label("joint: Gram 1 of the shard");
  if (e == cudaSuccess) e = gram_tall_sum(w.b.Yh, w.b.Yl, n, r, w.b, W_partial, w.status, st);
  return from_cuda(e);
}

loract_status_t loract_joint_orthonormalise(const loract_desc_t* desc, int32_t round, const float* W_sum,
                                            float* W_next_partial, void* U_local, void* ws, size_t ws_bytes,
                                            void* stream) {
  loract_status_t s = check_joint(desc);
  if (s != LORACT_OK) return s;
  if (round != 0 && round != 1) return LORACT_ERR_INVALID_ARG;
  if (!W_sum || !ws || (round == 0 && !W_next_partial) || (round == 1 && !U_local)) return LORACT_ERR_INVALID_ARG;
  if (misaligned(W_sum) || (round == 0 && misaligned(W_next_partial)) || (round == 1 && misaligned(U_local)) ||
      ((uintptr_t)ws & 255))
    return LORACT_ERR_ALIGNMENT;
  JointWs w;
  Plan plan;
  if (ws_bytes < carve_joint(ws, desc, &w, &plan)) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  const int r = desc->rank, n = (int)desc->n_tokens;
  trace_label(round ? "joint: small block 3" : "joint: small block 2");
  cudaError_t e = factor_matrix(W_sum, r, round ? kShiftSecond : kShiftFirstMean, w.b, w.status, st);
  trace_label(round ? "joint: apply L^-T 2" : "joint: apply L^-T 1");
  if (round == 0) {
    if (e == cudaSuccess) e = apply_linv(w.b.Yh, w.b.Yl, n, r, w.b, w.b.Qh, w.b.Ql, w.status, st);
    trace_label("joint: Gram 2 of the shard");
    if (e == cudaSuccess) e = gram_tall_sum(w.b.Qh, w.b.Ql, n, r, w.b, W_next_partial, w.status, st);
  } else {
    if (e == cudaSuccess) e = apply_linv(w.b.Qh, w.b.Ql, n, r, w.b, U_local, nullptr, w.status, st);
  }
  return from_cuda(e);
}

loract_status_t loract_joint_project(const loract_desc_t* desc, const void* U_local, const void* X_local,
                                     float* V_partial, void* ws, size_t ws_bytes, void* stream) {
  loract_status_t s = check_joint(desc);
  if (s != LORACT_OK) return s;
  if (!U_local || !X_local || !V_partial || !ws) return LORACT_ERR_INVALID_ARG;
  if (misaligned(U_local) || misaligned(X_local) || misaligned(V_partial) || ((uintptr_t)ws & 255))
    return LORACT_ERR_ALIGNMENT;
  JointWs w;
  Plan plan;
  if (ws_bytes < carve_joint(ws, desc, &w, &plan)) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  cudaStream_t st = (cudaStream_t)stream;
  GemmDesc g;
  g.M = plan.l; g.N = (int)plan.d; g.K = (int)plan.n; g.a_mn = true; g.b_mn = true; g.lda = plan.l; g.ldb = desc->ldx;
  g.terms[0] = {U_local, X_local};
  g.ldc = plan.d; g.out = OUT_F32;
  trace_label("joint: pass 2 of the shard");
  if (w.b.splits_v <= 1) { g.C0 = V_partial; return from_cuda(run_gemm(g, w.status, st)); }
  g.C0 = w.b.v_partials; g.splits = w.b.splits_v; g.split_stride = (int64_t)plan.l * plan.d;
  cudaError_t e = run_gemm(g, w.status, st);
  if (e == cudaSuccess)
    e = reduce_partials_launch(w.b.v_partials, w.b.splits_v, g.split_stride, g.split_stride, V_partial, nullptr, st);
  return from_cuda(e);
}

loract_status_t loract_joint_finish(const loract_desc_t* desc, const float* V_sum, void* V, void* stream) {
  loract_status_t s = check_joint(desc);
  if (s != LORACT_OK) return s;
  if (!V_sum || !V) return LORACT_ERR_INVALID_ARG;
  if (misaligned(V_sum) || misaligned(V)) return LORACT_ERR_ALIGNMENT;
  const int64_t count = (int64_t)desc->rank * desc->d;
  return from_cuda(reduce_partials_launch(V_sum, 1, 0, count, nullptr, (__nv_bfloat16*)V, (cudaStream_t)stream));
}

size_t loract_rsvd_workspace_bytes(const loract_desc_t* desc, int32_t oversample) {
  if (check_desc(desc) != LORACT_OK || desc->dtype != LORACT_BF16) return 0;
  const int l = desc->rank + oversample;
  if (oversample < 0 || oversample > 128 || l % 8 || l > 640 || l > desc->n_tokens || l > desc->d) return 0;
  Plan plan = make_plan(desc->n_tokens, desc->d, l, true);
  Carver c(nullptr);
  c.take(256);
  c.take((size_t)l * desc->d * 2);  // test matrix
  c.take((size_t)l * desc->d * 2);  // Q^T X of the power iterations, before it is preconditioned
  BasisWs b;
  carve_basis(c, plan, &b);
  return c.off;
}

loract_status_t loract_rsvd(const loract_desc_t* desc, int32_t oversample, const void* X, void* Uq, void* B,
                            void* ws, size_t ws_bytes, void* stream) {
  // t of Algorithm 1 is taken from desc->power_iters here, so validate a copy with t = 0
  if (!desc) return LORACT_ERR_INVALID_ARG;
  loract_desc_t d0 = *desc;
  d0.power_iters = 0;
  loract_status_t s = check_desc(&d0);
  if (s != LORACT_OK) return s;
  if (desc->dtype != LORACT_BF16) return LORACT_ERR_UNSUPPORTED;
  if (desc->power_iters < 0 || desc->power_iters > 8) return LORACT_ERR_INVALID_ARG;
  const size_t need = loract_rsvd_workspace_bytes(&d0, oversample);
  if (need == 0) return LORACT_ERR_INVALID_ARG;
  if (!X || !Uq || !B || !ws) return LORACT_ERR_INVALID_ARG;
  if (misaligned(X) || misaligned(Uq) || misaligned(B) || ((uintptr_t)ws & 255)) return LORACT_ERR_ALIGNMENT;
  if (ws_bytes < need) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  const int l = desc->rank + oversample;
  Plan plan = make_plan(desc->n_tokens, desc->d, l, true);
  Carver c(ws);
  uint32_t* status = (uint32_t*)c.take(256);
  __nv_bfloat16* Om = (__nv_bfloat16*)c.take((size_t)l * desc->d * 2);
  __nv_bfloat16* Tq = (__nv_bfloat16*)c.take((size_t)l * desc->d * 2);
  BasisWs b;
  carve_basis(c, plan, &b);
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemsetAsync(status, 0, 4, st);
  if (e == cudaSuccess) e = gaussian_rows_launch(desc->seed, desc->call_id, l, desc->d, Om, st);
  if (e == cudaSuccess) e = range_basis(X, desc->ldx, plan, Om, Uq, b, status, st);
  for (int it = 0; it < desc->power_iters && e == cudaSuccess; ++it) {
    // Y = X (X^T Q): X^T Q is kept transposed (l x d), which is exactly the test-matrix layout.  Its rows are
    // brought close to orthonormal first (same row space, so the same range), as in loract_compress: the
    // sketch would otherwise carry the cube of X's spectrum into a Gram matrix.
    e = project(Uq, X, desc->ldx, plan, Tq, b, status, st);
    if (e == cudaSuccess) e = precondition_rows(Tq, l, desc->d, true, Om, b, status, st);
    if (e == cudaSuccess) e = range_basis(X, desc->ldx, plan, Om, Uq, b, status, st);
  }
  if (e == cudaSuccess) e = project(Uq, X, desc->ldx, plan, B, b, status, st);
  return from_cuda(e);
}

loract_status_t loract_read_device_status(const void* ws, uint32_t* out_host, void* stream) {
  if (!ws || !out_host) return LORACT_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  cudaError_t e = cudaMemcpyAsync(out_host, ws, 4, cudaMemcpyDeviceToHost, st);
  if (e == cudaSuccess) e = cudaStreamSynchronize(st);
  return from_cuda(e);
}

const char* loract_status_string(loract_status_t s) {
  switch (s) {
    case LORACT_OK: return "ok";
    case LORACT_ERR_INVALID_ARG: return "invalid argument";
    case LORACT_ERR_UNSUPPORTED: return "unsupported";
    case LORACT_ERR_ALIGNMENT: return "misaligned pointer or stride";
    case LORACT_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LORACT_ERR_CUDA: return "CUDA error";
    case LORACT_ERR_NUMERIC: return "numerical breakdown";
    case LORACT_ERR_TIMEOUT: return "device wait expired";
  }
  return "unknown status";
}

loract_status_t loract_status_from_device_word(uint32_t word) {
  if (word & LORACT_DEV_WAIT_EXPIRED) return LORACT_ERR_TIMEOUT;
  if (word & (LORACT_DEV_NONFINITE | LORACT_DEV_SAMPLER_SHORT)) return LORACT_ERR_NUMERIC;
  return LORACT_OK;   // a clamped pivot alone is a warning: the factors are valid
}

loract_status_t loract_debug_wait_expiry(int32_t which, uint64_t limit_ns, uint32_t* status_word, void* stream) {
  if (!status_word || limit_ns == 0 || limit_ns > 100000000ull) return LORACT_ERR_INVALID_ARG;   // 100 ms at most
  cudaStream_t st = (cudaStream_t)stream;
  if (which == 0) return from_cuda(gemm_tc_wait_probe_launch(status_word, limit_ns, st));
  if (which == 1) return from_cuda(small_block_cluster_wait_probe_launch(status_word, limit_ns, st));
  return LORACT_ERR_INVALID_ARG;
}

uint64_t loract_kernel_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

loract_status_t loract_debug_gemm(int32_t M, int32_t N, int32_t K, int32_t a_mn, int32_t b_mn,
                                  const void* const* A, int64_t lda, const void* const* B, int64_t ldb,
                                  int32_t a_type, int32_t b_type, int32_t n_terms, int32_t out_mode, void* C0,
                                  void* C1, int64_t ldc, int32_t splits, int64_t split_stride, int32_t acc64,
                                  int32_t engine, uint32_t* status_word, void* stream) {
  return loract_debug_gemm_halved(M, N, K, a_mn, b_mn, A, lda, B, ldb, a_type, b_type, n_terms, 0, out_mode, C0, C1,
                                  ldc, splits, split_stride, acc64, engine, status_word, stream);
}

loract_status_t loract_debug_reduce_sym(const float* partials, int32_t n_partials, int64_t stride, int32_t r,
                                        float* out, void* stream) {
  if (!partials || !out || n_partials < 1 || r < 1) return LORACT_ERR_INVALID_ARG;
  return from_cuda(reduce_sym_launch(partials, n_partials, stride, r, out, (cudaStream_t)stream));
}

loract_status_t loract_debug_gemm_halved(int32_t M, int32_t N, int32_t K, int32_t a_mn, int32_t b_mn,
                                         const void* const* A, int64_t lda, const void* const* B, int64_t ldb,
                                         int32_t a_type, int32_t b_type, int32_t n_terms, int32_t halve_at_term,
                                         int32_t out_mode, void* C0, void* C1, int64_t ldc, int32_t splits,
                                         int64_t split_stride, int32_t acc64, int32_t engine, uint32_t* status_word,
                                         void* stream) {
  if (!A || !B || !C0 || n_terms < 1 || n_terms > 3 || M < 1 || N < 1 || K < 1) return LORACT_ERR_INVALID_ARG;
  if (halve_at_term < 0 || halve_at_term >= n_terms) return LORACT_ERR_INVALID_ARG;
  GemmDesc g;
  g.M = M; g.N = N; g.K = K; g.a_mn = a_mn != 0; g.b_mn = b_mn != 0; g.lda = lda; g.ldb = ldb;
  g.a_type = a_type; g.b_type = b_type; g.n_terms = n_terms;
  for (int t = 0; t < n_terms; ++t) g.terms[t] = {A[t], B[t]};
  g.out = out_mode; g.C0 = C0; g.C1 = C1; g.ldc = ldc; g.splits = splits < 1 ? 1 : splits;
  g.split_stride = split_stride; g.acc64 = acc64 != 0;
  g.halve_at_term = halve_at_term;
  if (engine == 1) {
    if (!gemm_tc_supported(g)) return LORACT_ERR_UNSUPPORTED;
    return from_cuda(gemm_tc_launch(g, status_word, (cudaStream_t)stream));
  }
  return from_cuda(gemm_simt_launch(g, (cudaStream_t)stream));
}

loract_status_t loract_debug_project(const loract_desc_t* desc, const void* U, const void* X, void* V, void* ws,
                                     size_t ws_bytes, void* stream) {
  loract_status_t s = check_desc(desc);
  if (s != LORACT_OK) return s;
  if (!U || !X || !V || !ws) return LORACT_ERR_INVALID_ARG;
  CompressWs w;
  Plan plan;
  const size_t need = carve_compress(ws, desc, /*with_A=*/false, &w, &plan);
  if (ws_bytes < need) return LORACT_ERR_WORKSPACE_TOO_SMALL;
  return from_cuda(project(U, X, desc->ldx, plan, V, w.b, w.status, (cudaStream_t)stream));
}

void loract_debug_trace_begin(void* stream) {
  g_trace_used = 0;
  g_trace_names.clear();
  g_trace_open = true;
  trace_label("");
  cudaEvent_t e = trace_event();
  if (e) cudaEventRecord(e, (cudaStream_t)stream);
}

int32_t loract_debug_trace_end(void* stream, char* names, float* micros, int32_t max_entries) {
  g_trace_open = false;
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess) return -1;
  int32_t n = 0;
  for (size_t i = 0; i + 1 < g_trace_used && n < max_entries; ++i, ++n) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, g_trace_events[i], g_trace_events[i + 1]);
    micros[n] = ms * 1000.f;
    std::strncpy(names + (size_t)n * 64, g_trace_names[i].c_str(), 63);
    names[(size_t)n * 64 + 63] = 0;
  }
  return n;
}

void loract_debug_set_pair_mode(int32_t on) { gemm_tc_set_pair_mode(on); }

loract_status_t loract_debug_round_gate(const float* W, const void* linv_hi, int32_t r, float threshold,
                                        const uint32_t* status_word, uint32_t* words, void* stream) {
  if (!W || !linv_hi || !words) return LORACT_ERR_INVALID_ARG;
  return from_cuda(round_gate_launch(W, (const __nv_bfloat16*)linv_hi, r, threshold, status_word, words,
                                     (cudaStream_t)stream));
}

void loract_debug_set_round_gate(float threshold) {
  g_round_gate.store(threshold == 0.f ? kRoundGateDefault : threshold);
}

int32_t loract_debug_last_cuda_error(void) { return g_last_cuda_error.load(std::memory_order_relaxed); }

loract_status_t loract_debug_small_block(int32_t r, const void* partials, int32_t partial_f64, int32_t n_partials,
                                         int64_t partial_stride, int32_t use_f64, float shift_rel, void* scratch,
                                         float* linv_f32, void* linv_hi, void* linv_lo, uint32_t* status_word,
                                         void* stream) {
  if (r < 16 || r > 640 || r % 8 || !partials || !scratch || n_partials < 1) return LORACT_ERR_INVALID_ARG;
  SmallBlockArgs a;
  a.r = r; a.partials = partials; a.partial_type = partial_f64 ? ELEM_F64 : ELEM_F32;
  a.n_partials = n_partials; a.partial_stride = partial_stride; a.use_f64 = use_f64 != 0;
  a.scratch = scratch; a.shift_rel = shift_rel; a.linv_f32 = linv_f32;
  a.linv_hi = (__nv_bfloat16*)linv_hi; a.linv_lo = (__nv_bfloat16*)linv_lo; a.dev_status = status_word;
  return from_cuda(small_block_launch(a, (cudaStream_t)stream));
}

}  // extern "C"

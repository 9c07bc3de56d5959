// CPU oracle for the EFCP / Sparse M-FAC step.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain restatement of what one optimizer step computes.
// It exists so that the CUDA library can be compared against something written
// straight from the paper's formulas.  It shares no code, header, table or
// helper with the CUDA path and must never be linked into, imported by or
// called from the product library or its Python binding.  Only the tests, the
// smoke check and the CPU-baseline leg of the benchmark may use it.
//
// What each function follows:
//   * step 1-3 (error feedback, Top-k compress, residual): Algorithm 1, the error-feedback, compression and error-update statements
//     and the "Overview" paragraph of Section 3.
//   * Top-k: Section 3.1 (keep the k largest-magnitude entries as index/value
//     pairs).  Global over d, ties go to the lower index, pairs stored by
//     ascending index; magnitude order is the unsigned order of the IEEE bit
//     pattern with the sign bit cleared.
//   * ring buffer G=(I,V): Section 2.1 (ring buffer of the last m gradients) and
//     Section 3.1 "Sparsity format for G" (row replacement).
//   * scalar products / Gram matrix: Section 2.1 "Scalar Products (SP)":
//     S = G G^T, row and column i replaced by G g when row i is replaced.
//   * inverse-Fisher-vector product: Section 2.1, F = lambda I + (1/m) sum g g^T,
//     Eq. (2): F^-1 x = x/lambda - sum_k c_k g_k.  The coefficients are obtained
//     from the Woodbury identity
//        (lambda I + (1/m) G^T G)^-1 = I/lambda - (1/lambda) G^T (m lambda I + G G^T)^-1 G,
//     i.e. c = (1/lambda) (m lambda I + S)^-1 (G x), solved by a Cholesky
//     factorisation in fp64.  efcp_ref_wsm_coef carries the literal
//     Woodbury-Sherman-Morrison rank-one recursion of Section 2.1 as a second,
//     independent route to the same coefficients.
//   * linear combination of gradients: Section 2.1 "LCG" and Eq. (2).
//   * optional bfloat16 window values: Section 3.1 "Format for V".  Reading taken (the paper
//     only says the optimizer still converges with bfloat16 values): Compress returns the
//     selected values rounded to bfloat16, and the error update of Algorithm 1 is applied to that c,
//     so the rounding residue is fed back like any other compression error.
//
// Precision: the state (error buffer, window) is fp32 exactly as the method
// defines it (one IEEE round-to-nearest add per coordinate, no fused multiply
// add, no flush-to-zero).  Everything from the scalar products on is fp64 with
// a single final rounding of the update to fp32.
//
// Parity pins (tests not marked gpu): brute-force dense d x d solves on tiny
// problems, the invariant a == e_new + dens(c) bit for bit, Top-k against a
// full stable sort, the closed forms for m = 1 and for rows with disjoint
// supports, the large-lambda limit, the WSM recursion against the Cholesky
// route, k == d (dense M-FAC); the bfloat16 rounding against a library conversion
// and hand-made tie cases.  No numeric example is printed in the paper, so
// beyond those pins the values are "parity unpinned".
//
// Threads: OpenMP is used only on loops whose every output element is produced
// by one thread running the same sequential inner loop, so results do not
// depend on the thread count.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <new>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr uint32_t kFlagRhsAccumulator = 1u;  // x = a_t instead of x = dens(c_t)
constexpr uint32_t kFlagValuesBf16 = 2u;      // kept values are rounded to bfloat16

// fp32 -> bfloat16 -> fp32, round to nearest, ties to even (the bfloat16 format of Section
// 3.1 "Format for V": the upper 16 bits of an IEEE fp32).  NaN stays NaN.
inline float round_to_bf16(float v) {
  uint32_t b;
  std::memcpy(&b, &v, 4);
  if ((b & 0x7FFFFFFFu) > 0x7F800000u) {
    b |= 0x00400000u;  // quiet NaN, payload truncated
    b &= 0xFFFF0000u;
  } else {
    const uint32_t lsb = (b >> 16) & 1u;
    b += 0x7FFFu + lsb;
    b &= 0xFFFF0000u;
  }
  float r;
  std::memcpy(&r, &b, 4);
  return r;
}

inline uint32_t magnitude_key(float v) {
  uint32_t b;
  std::memcpy(&b, &v, 4);
  return b & 0x7FFFFFFFu;
}

struct Oracle {
  int64_t d = 0;
  int32_t m = 0;
  int64_t k = 0;
  float lambda = 0.f;
  uint32_t flags = 0;
  int64_t block = 0;  // > 0: Top-k is applied per block of this many coordinates
  int64_t k_req = 0;  // the k the caller asked for (k is the row length actually kept)
  int64_t t = 0;  // number of completed steps
  std::vector<float> e;      // error feedback buffer (xi), d
  std::vector<float> a;      // accumulator of the last step, d
  std::vector<int32_t> I;    // m*k indices
  std::vector<float> V;      // m*k values
  std::vector<double> S;     // m*m Gram matrix
  std::vector<double> p;     // m, G x of the last step
  std::vector<double> coef;  // m, Eq. (2) coefficients of the last step
  std::vector<double> L;     // m*m Cholesky workspace
  std::vector<double> acc;   // d, fp64 accumulator for the update
  std::vector<double> xd;    // d, dense right-hand side in fp64
  std::vector<uint64_t> order;  // d, Top-k workspace
};

// Composite sort word: larger word = earlier in the (key descending, index
// ascending) order.
inline uint64_t order_word(uint32_t key, int64_t j) {
  return (uint64_t(key) << 32) | uint64_t(0xFFFFFFFFu - uint32_t(j));
}

// Top-k by selection: the k largest composite words are, by construction of
// the word, the first k entries of a sort by (|a| descending, index ascending).
void topk_select(const float* a, int64_t d, int64_t k, std::vector<uint64_t>& w,
                 int32_t* idx, float* val) {
  w.resize(size_t(d));
  for (int64_t j = 0; j < d; ++j) w[size_t(j)] = order_word(magnitude_key(a[j]), j);
  if (k < d) {
    std::nth_element(w.begin(), w.begin() + k, w.end(), std::greater<uint64_t>());
  }
  std::vector<int32_t> sel(static_cast<size_t>(k));
  for (int64_t r = 0; r < k; ++r)
    sel[size_t(r)] = int32_t(0xFFFFFFFFu - uint32_t(w[size_t(r)] & 0xFFFFFFFFu));
  std::sort(sel.begin(), sel.end());
  for (int64_t r = 0; r < k; ++r) {
    idx[r] = sel[size_t(r)];
    val[r] = a[sel[size_t(r)]];
  }
}

// Cholesky A = L L^T (lower, row-major, n x n).  Column by column; within a
// column every row is independent.  Returns the index of the first
// non-positive pivot + 1, or 0 on success.
int cholesky_lower(const double* A, double* L, int n) {
  for (int j = 0; j < n; ++j) {
    double s = A[size_t(j) * n + j];
    const double* Lj = L + size_t(j) * n;
    for (int q = 0; q < j; ++q) s -= Lj[q] * Lj[q];
    if (!(s > 0.0)) return j + 1;
    const double piv = std::sqrt(s);
    L[size_t(j) * n + j] = piv;
#pragma omp parallel for schedule(static)
    for (int i = j + 1; i < n; ++i) {
      const double* Li = L + size_t(i) * n;
      double v = A[size_t(i) * n + j];
      for (int q = 0; q < j; ++q) v -= Li[q] * Lj[q];
      L[size_t(i) * n + j] = v / piv;
    }
  }
  return 0;
}

// Solve L L^T y = b.
void cholesky_solve(const double* L, int n, const double* b, double* y) {
  std::vector<double> f(static_cast<size_t>(n));
  for (int i = 0; i < n; ++i) {
    double v = b[i];
    const double* Li = L + size_t(i) * n;
    for (int q = 0; q < i; ++q) v -= Li[q] * f[size_t(q)];
    f[size_t(i)] = v / Li[i];
  }
  for (int i = n - 1; i >= 0; --i) {
    double v = f[size_t(i)];
    for (int q = i + 1; q < n; ++q) v -= L[size_t(q) * n + i] * y[q];
    y[i] = v / L[size_t(i) * n + i];
  }
}

}  // namespace

extern "C" {

struct efcp_ref;  // opaque for callers

// Element-wise fp32 -> bfloat16 -> fp32 (round to nearest even), for the pins.
void efcp_ref_round_bf16(const float* in, float* out, int64_t n) {
  for (int64_t j = 0; j < n; ++j) out[j] = round_to_bf16(in[j]);
}

// Exact Top-k of |a| (ties to the lower index), pairs in ascending index order.
int efcp_ref_topk(const float* a, int64_t d, int64_t k, int32_t* idx, float* val) {
  if (!a || !idx || !val || d < 1 || k < 1 || k > d || d >= (int64_t(1) << 31)) return -1;
  std::vector<uint64_t> w;
  topk_select(a, d, k, w, idx, val);
  return 0;
}

// The same result by the definition itself: a stable sort of all d positions by
// magnitude key descending (stability keeps the lower index first among equal
// keys), the first k taken, then put in ascending index order.
int efcp_ref_topk_fullsort(const float* a, int64_t d, int64_t k, int32_t* idx, float* val) {
  if (!a || !idx || !val || d < 1 || k < 1 || k > d || d >= (int64_t(1) << 31)) return -1;
  std::vector<int32_t> pos(static_cast<size_t>(d));
  for (int64_t j = 0; j < d; ++j) pos[size_t(j)] = int32_t(j);
  std::stable_sort(pos.begin(), pos.end(), [a](int32_t x, int32_t y) {
    return magnitude_key(a[x]) > magnitude_key(a[y]);
  });
  std::vector<int32_t> sel(pos.begin(), pos.begin() + k);
  std::sort(sel.begin(), sel.end());
  for (int64_t r = 0; r < k; ++r) {
    idx[r] = sel[size_t(r)];
    val[r] = a[sel[size_t(r)]];
  }
  return 0;
}

// Eq. (2) coefficients through the Woodbury identity:
//   coef = (1/lambda) (m lambda I + S)^-1 p           (fp64 Cholesky)
// S is m x m row-major.  Returns 0, or j+1 when pivot j is not positive.
int efcp_ref_woodbury_coef(const double* S, const double* p, int32_t m, double lambda,
                           double* coef) {
  if (!S || !p || !coef || m < 1 || !(lambda > 0)) return -1;
  std::vector<double> A(size_t(m) * m), L(size_t(m) * m, 0.0), y(static_cast<size_t>(m));
  for (int i = 0; i < m; ++i)
    for (int j = 0; j < m; ++j)
      A[size_t(i) * m + j] = S[size_t(i) * m + j] + (i == j ? double(m) * lambda : 0.0);
  int bad = cholesky_lower(A.data(), L.data(), m);
  if (bad) return bad;
  cholesky_solve(L.data(), m, p, y.data());
  for (int i = 0; i < m; ++i) coef[i] = y[size_t(i)] / lambda;
  return 0;
}

// Eq. (2) coefficients through the literal rank-one recursion of Section 2.1:
//   F_0 = lambda I,  F_j = F_{j-1} + (1/m) g_j g_j^T,
//   F_j^-1 x = F_{j-1}^-1 x - v_j (v_j^T x) / (m + g_j^T v_j),   v_j = F_{j-1}^-1 g_j.
// Every v_j is a combination of the window rows, v_j = sum_l beta[j][l] g_l,
// so only the scalar products S = G G^T and p = G x are needed.
int efcp_ref_wsm_coef(const double* S, const double* p, int32_t m, double lambda,
                      double* coef) {
  if (!S || !p || !coef || m < 1 || !(lambda > 0)) return -1;
  const size_t n = size_t(m);
  std::vector<double> beta(n * n, 0.0), D(n, 0.0), vg(n, 0.0);
  for (int j = 0; j < m; ++j) {
    // vg[i] = v_i^T g_j for i < j
    for (int i = 0; i < j; ++i) {
      double s = 0.0;
      for (int l = 0; l <= i; ++l) s += beta[size_t(i) * n + l] * S[size_t(l) * n + j];
      vg[size_t(i)] = s;
    }
    // v_j = g_j/lambda - sum_{i<j} v_i (v_i^T g_j) / D_i
    double* bj = &beta[size_t(j) * n];
    bj[j] = 1.0 / lambda;
    for (int i = 0; i < j; ++i) {
      const double f = vg[size_t(i)] / D[size_t(i)];
      for (int l = 0; l <= i; ++l) bj[l] -= f * beta[size_t(i) * n + l];
    }
    double gv = 0.0;
    for (int l = 0; l <= j; ++l) gv += bj[l] * S[size_t(l) * n + j];
    D[size_t(j)] = double(m) + gv;
  }
  for (int l = 0; l < m; ++l) coef[l] = 0.0;
  for (int j = 0; j < m; ++j) {
    double q = 0.0;
    for (int l = 0; l <= j; ++l) q += beta[size_t(j) * n + l] * p[l];
    const double f = q / D[size_t(j)];
    for (int l = 0; l <= j; ++l) coef[l] += f * beta[size_t(j) * n + l];
  }
  return 0;
}

// Entries block-wise Top-k keeps in a block of `len` coordinates at density k/d:
// ceil(len * k / d) (Section 3.1 "Sparsity Pattern": ceil(B / 100) at 1 %).
int64_t efcp_ref_block_count(int64_t len, int64_t k, int64_t d) { return (len * k + d - 1) / d; }

// block > 0: Top-k applied in blocks of `block` coordinates (Section 3.1, "Sparsity
// Pattern"); every row then holds the sum of the per-block counts, see
// efcp_ref_row_length.  block == 0: one global Top-k of k entries.
int efcp_ref_create_blockwise(efcp_ref** out, int64_t d, int32_t m, int64_t k, float lambda,
                              uint32_t flags, int64_t block) {
  if (!out) return -1;
  *out = nullptr;
  if (d < 1 || m < 1 || k < 1 || k > d || d >= (int64_t(1) << 31) || block < 0) return -1;
  if (!(lambda > 0.f) || !std::isfinite(lambda)) return -1;
  Oracle* o = new (std::nothrow) Oracle();
  if (!o) return -2;
  try {
    o->k_req = k;
    o->block = block;
    if (block > 0) {
      int64_t total = 0;
      for (int64_t b0 = 0; b0 < d; b0 += block)
        total += efcp_ref_block_count(std::min(block, d - b0), k, d);
      k = total;
    }
    o->d = d; o->m = m; o->k = k; o->lambda = lambda; o->flags = flags;
    o->e.assign(size_t(d), 0.f);
    o->a.assign(size_t(d), 0.f);
    o->I.resize(size_t(m) * size_t(k));
    o->V.assign(size_t(m) * size_t(k), 0.f);
    // A row that has not been written yet is a zero gradient: values 0 at the
    // first k coordinates.
    for (int32_t r = 0; r < m; ++r)
      for (int64_t j = 0; j < k; ++j) o->I[size_t(r) * size_t(k) + size_t(j)] = int32_t(j);
    o->S.assign(size_t(m) * m, 0.0);
    o->p.assign(size_t(m), 0.0);
    o->coef.assign(size_t(m), 0.0);
    o->L.assign(size_t(m) * m, 0.0);
    o->acc.assign(size_t(d), 0.0);
    o->xd.assign(size_t(d), 0.0);
  } catch (const std::bad_alloc&) {
    delete o;
    return -2;
  }
  *out = reinterpret_cast<efcp_ref*>(o);
  return 0;
}

int efcp_ref_create(efcp_ref** out, int64_t d, int32_t m, int64_t k, float lambda,
                    uint32_t flags) {
  return efcp_ref_create_blockwise(out, d, m, k, lambda, flags, 0);
}

// Entries per row: k for global Top-k, the sum of the per-block counts otherwise.
int64_t efcp_ref_row_length(efcp_ref* h) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  return o ? o->k : -1;
}

void efcp_ref_destroy(efcp_ref* h) { delete reinterpret_cast<Oracle*>(h); }

// One optimizer step.  grad and update are host arrays of d floats.
// Returns 0, or a positive pivot index + 1 if the Cholesky factorisation met a
// non-positive pivot.
int efcp_ref_step(efcp_ref* h, const float* grad, float* update) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !grad || !update) return -1;
  const int64_t d = o->d, k = o->k;
  const int32_t m = o->m;
  const double lambda = double(o->lambda);

  // Algorithm 1, error feedback: a = xi + g, one fp32 add per coordinate.
  // (built with -ffp-contract=off and without fast-math.)
  for (int64_t j = 0; j < d; ++j) o->a[size_t(j)] = o->e[size_t(j)] + grad[j];

  // Algorithm 1, compression: c = TopK(a); the row goes into ring slot i.
  const int32_t i = int32_t(o->t % m);
  int32_t* idx = &o->I[size_t(i) * size_t(k)];
  float* val = &o->V[size_t(i) * size_t(k)];
  if (o->block > 0) {
    // Section 3.1 "Sparsity Pattern": an exact Top-k inside every block of `block`
    // coordinates; the blocks follow one another, so the row stays in ascending order.
    int64_t pos = 0;
    for (int64_t b0 = 0; b0 < d; b0 += o->block) {
      const int64_t len = std::min(o->block, d - b0);
      const int64_t c = efcp_ref_block_count(len, o->k_req, d);
      topk_select(o->a.data() + b0, len, c, o->order, idx + pos, val + pos);
      for (int64_t r = 0; r < c; ++r) idx[pos + r] += int32_t(b0);
      pos += c;
    }
  } else {
    topk_select(o->a.data(), d, k, o->order, idx, val);
  }

  // Section 3.1 "Format for V" (optional): the window holds bfloat16 values, so c is the
  // selection with every value rounded to bfloat16.
  if (o->flags & kFlagValuesBf16)
    for (int64_t r = 0; r < k; ++r) val[r] = round_to_bf16(val[r]);

  // Algorithm 1, error update: xi = a - c.  A kept coordinate becomes literally +0 (what a - a
  // is for every finite a; a non-finite a would give NaN, and the method defines the kept
  // coordinate as removed from the error); with rounded values the rounding residue
  // a - bf16(a) (exact in fp32) stays in the error buffer.
  o->e = o->a;
  if (o->flags & kFlagValuesBf16) {
    for (int64_t r = 0; r < k; ++r)
      o->e[size_t(idx[r])] = o->a[size_t(idx[r])] - val[r];
  } else {
    for (int64_t r = 0; r < k; ++r) o->e[size_t(idx[r])] = 0.0f;
  }
  o->t += 1;

  // Right-hand side x of the inverse-Fisher-vector product.
  std::fill(o->xd.begin(), o->xd.end(), 0.0);
  std::vector<double> cd;  // dens(c) in fp64 when x = a (needed for the Gram row)
  if (o->flags & kFlagRhsAccumulator) {
    cd.assign(size_t(d), 0.0);
    for (int64_t r = 0; r < k; ++r) cd[size_t(idx[r])] = double(val[r]);
    for (int64_t j = 0; j < d; ++j) o->xd[size_t(j)] = double(o->a[size_t(j)]);
  } else {
    for (int64_t r = 0; r < k; ++r) o->xd[size_t(idx[r])] = double(val[r]);
  }
  const double* crow = (o->flags & kFlagRhsAccumulator) ? cd.data() : o->xd.data();

  // Scalar products: row and column i of S become G c; p = G x.
  std::vector<double> delta(static_cast<size_t>(m));
#pragma omp parallel for schedule(static)
  for (int32_t r = 0; r < m; ++r) {
    const int32_t* Ir = &o->I[size_t(r) * size_t(k)];
    const float* Vr = &o->V[size_t(r) * size_t(k)];
    double s = 0.0, q = 0.0;
    for (int64_t j = 0; j < k; ++j) {
      s += double(Vr[j]) * crow[size_t(Ir[j])];
      q += double(Vr[j]) * o->xd[size_t(Ir[j])];
    }
    delta[size_t(r)] = s;
    o->p[size_t(r)] = q;
  }
  for (int32_t r = 0; r < m; ++r) {
    o->S[size_t(i) * m + r] = delta[size_t(r)];
    o->S[size_t(r) * m + i] = delta[size_t(r)];
  }

  // Coefficients of Eq. (2): (m lambda I + S) y = p, coef = y / lambda.
  int bad = efcp_ref_woodbury_coef(o->S.data(), o->p.data(), m, lambda, o->coef.data());
  if (bad) return bad;

  // Eq. (2): u = x / lambda - sum_r coef_r row_r, accumulated in fp64.
  for (int64_t j = 0; j < d; ++j) o->acc[size_t(j)] = o->xd[size_t(j)] / lambda;
  for (int32_t r = 0; r < m; ++r) {
    const int32_t* Ir = &o->I[size_t(r) * size_t(k)];
    const float* Vr = &o->V[size_t(r) * size_t(k)];
    const double cr = o->coef[size_t(r)];
    for (int64_t j = 0; j < k; ++j) o->acc[size_t(Ir[j])] -= cr * double(Vr[j]);
  }
  for (int64_t j = 0; j < d; ++j) update[j] = float(o->acc[size_t(j)]);
  return 0;
}

// The same update through the cancellation-free form that holds when x is row
// i of the window (x = dens(c_t)):  u = m G^T (m lambda I + S)^-1 e_i.
// Uses the state left by the last efcp_ref_step; writes d floats.
int efcp_ref_update_rowform(efcp_ref* h, float* update) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !update || o->t < 1 || (o->flags & kFlagRhsAccumulator)) return -1;
  const int32_t m = o->m;
  const int64_t d = o->d, k = o->k;
  const int32_t i = int32_t((o->t - 1) % m);
  std::vector<double> ei(size_t(m), 0.0), w(static_cast<size_t>(m));
  ei[size_t(i)] = double(m);  // (1/lambda)(m lambda I + S)^-1 (lambda m e_i)
  int bad = efcp_ref_woodbury_coef(o->S.data(), ei.data(), m, double(o->lambda), w.data());
  if (bad) return bad;
  for (int32_t r = 0; r < m; ++r) w[size_t(r)] *= double(o->lambda);
  std::vector<double> acc(size_t(d), 0.0);
  for (int32_t r = 0; r < m; ++r) {
    const int32_t* Ir = &o->I[size_t(r) * size_t(k)];
    const float* Vr = &o->V[size_t(r) * size_t(k)];
    for (int64_t j = 0; j < k; ++j) acc[size_t(Ir[j])] += w[size_t(r)] * double(Vr[j]);
  }
  for (int64_t j = 0; j < d; ++j) update[j] = float(acc[size_t(j)]);
  return 0;
}

// S recomputed from the window as G G^T (fp64), for checking the row/column
// replacement bookkeeping.  out is m*m row-major.
int efcp_ref_gram_full(efcp_ref* h, double* out) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !out) return -1;
  const int32_t m = o->m;
  const int64_t d = o->d, k = o->k;
  std::vector<double> dense(size_t(d), 0.0);
  for (int32_t s = 0; s < m; ++s) {
    const int32_t* Is = &o->I[size_t(s) * size_t(k)];
    const float* Vs = &o->V[size_t(s) * size_t(k)];
    for (int64_t j = 0; j < k; ++j) dense[size_t(Is[j])] = double(Vs[j]);
    for (int32_t r = 0; r < m; ++r) {
      const int32_t* Ir = &o->I[size_t(r) * size_t(k)];
      const float* Vr = &o->V[size_t(r) * size_t(k)];
      double acc = 0.0;
      for (int64_t j = 0; j < k; ++j) acc += double(Vr[j]) * dense[size_t(Ir[j])];
      out[size_t(r) * m + s] = acc;
    }
    for (int64_t j = 0; j < k; ++j) dense[size_t(Is[j])] = 0.0;
  }
  return 0;
}

int64_t efcp_ref_step_count(efcp_ref* h) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  return o ? o->t : -1;
}
int efcp_ref_get_error(efcp_ref* h, float* out) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !out) return -1;
  std::memcpy(out, o->e.data(), size_t(o->d) * 4);
  return 0;
}
int efcp_ref_get_accumulator(efcp_ref* h, float* out) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !out) return -1;
  std::memcpy(out, o->a.data(), size_t(o->d) * 4);
  return 0;
}
int efcp_ref_get_row(efcp_ref* h, int32_t slot, int32_t* idx, float* val) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !idx || !val || slot < 0 || slot >= o->m) return -1;
  std::memcpy(idx, &o->I[size_t(slot) * size_t(o->k)], size_t(o->k) * 4);
  std::memcpy(val, &o->V[size_t(slot) * size_t(o->k)], size_t(o->k) * 4);
  return 0;
}
int efcp_ref_get_gram(efcp_ref* h, double* out) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !out) return -1;
  std::memcpy(out, o->S.data(), size_t(o->m) * o->m * 8);
  return 0;
}
int efcp_ref_get_p(efcp_ref* h, double* out) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !out) return -1;
  std::memcpy(out, o->p.data(), size_t(o->m) * 8);
  return 0;
}
int efcp_ref_get_coef(efcp_ref* h, double* out) {
  Oracle* o = reinterpret_cast<Oracle*>(h);
  if (!o || !out) return -1;
  std::memcpy(out, o->coef.data(), size_t(o->m) * 8);
  return 0;
}
int efcp_ref_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Size of the OpenMP team for the calls that follow (timing the single-thread baseline);
// no result depends on it.
void efcp_ref_set_num_threads(int32_t n) {
#ifdef _OPENMP
  if (n >= 1) omp_set_num_threads(n);
#else
  (void)n;
#endif
}

}  // extern "C"

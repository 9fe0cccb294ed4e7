// WERSA float64 CPU oracle  --  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
//
// A plain, slow, obviously-correct restatement of the per-head WERSA attention
// operator (Wavelet-Enhanced Random Spectral Attention, arXiv 2507.08637) in
// double precision.  It shares no code with the CUDA library and must never be
// linked, imported or called by it; only the test-suite, the smoke check and
// the benchmark's CPU-baseline leg use it.
//
// Every function follows the paper's steps in the paper's order:
//   * mean-pooled query                    Sec. 3.1 step 4, Eq. 1
//   * gate: sigmoid(g(qbar)) * omega       Eq. 2, Eq. 3; Algorithm 1 (filters)
//   * Haar analysis, L levels              Appendix A Eqs. 19-20; Algorithm 2 (VectorizedDWT)
//   * per-scale filtering of coefficients  Sec. 3.1 step 5; Algorithm 2 (FilteredIDWT)
//   * Haar synthesis, trim                 Appendix A Eqs. 21-22; Algorithm 2 (VectorizedIDWT)
//   * random feature map                   Eq. 6 with Algorithm 1's max(beta, floor) and 1/sqrt(r)
//   * linear attention with normaliser     Eq. 7 / Sec. 3.1 step 8
// The backward pass is not written in the paper; it is the chain rule applied
// to those steps in reverse order, with d ReLU(a)/da = 1[a > 0].
//
// No blocking, fusion or reordering beyond those steps.  OpenMP is used only
// across independent (batch, head) slabs.
//
// Parity pins (tests/test_oracle_pins.py): perfect reconstruction, energy
// preservation, a hand-derived 4-sample worked example, block-mean identity,
// brute-force O(n^2) kernel attention, Monte-Carlo convergence to the
// arc-cosine kernel, convexity invariants, finite differences for every
// gradient.  The only claim with "parity unpinned" is the paper's statement
// that the feature map approximates the softmax kernel: it is not tested.

#include <cmath>
#include <cstddef>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

typedef std::vector<double> vec;

int next_pow2(int n) {
  int p = 1;
  while (p < n) p <<= 1;
  return p;
}

// Haar analysis of one (npad x d) signal, Algorithm 2 (VectorizedDWT), Eqs. 19-20.
// coeffs[0..L-1] = d_1..d_L  (d_l has npad/2^l rows), coeffs[L] = a_L.
void haar_dwt(const vec& xpad, int npad, int d, int L, std::vector<vec>& coeffs) {
  const double inv_sqrt2 = 1.0 / std::sqrt(2.0);
  coeffs.assign(L + 1, vec());
  vec approx = xpad;
  int rows = npad;
  for (int l = 1; l <= L; ++l) {
    int half = rows / 2;
    vec new_approx((size_t)half * d), detail((size_t)half * d);
    for (int k = 0; k < half; ++k)
      for (int c = 0; c < d; ++c) {
        double even = approx[(size_t)(2 * k) * d + c];
        double odd = approx[(size_t)(2 * k + 1) * d + c];
        new_approx[(size_t)k * d + c] = (even + odd) * inv_sqrt2;
        detail[(size_t)k * d + c] = (even - odd) * inv_sqrt2;
      }
    coeffs[l - 1].swap(detail);
    approx.swap(new_approx);
    rows = half;
  }
  coeffs[L].swap(approx);
}

// Haar synthesis, Algorithm 2 (VectorizedIDWT), Eqs. 21-22.  Returns npad rows.
void haar_idwt(const std::vector<vec>& coeffs, int npad, int d, int L, vec& out) {
  const double inv_sqrt2 = 1.0 / std::sqrt(2.0);
  vec approx = coeffs[L];
  int rows = npad >> L;
  for (int l = L; l >= 1; --l) {
    const vec& detail = coeffs[l - 1];
    vec next((size_t)rows * 2 * d);
    for (int k = 0; k < rows; ++k)
      for (int c = 0; c < d; ++c) {
        double a = approx[(size_t)k * d + c], dd = detail[(size_t)k * d + c];
        next[(size_t)(2 * k) * d + c] = (a + dd) * inv_sqrt2;
        next[(size_t)(2 * k + 1) * d + c] = (a - dd) * inv_sqrt2;
      }
    approx.swap(next);
    rows *= 2;
  }
  out.swap(approx);
}

// Zero-pad n rows to the next power of two (Algorithm 2, VectorizedDWT head).
void pad_rows(const double* x, int n, int d, int npad, vec& xpad) {
  xpad.assign((size_t)npad * d, 0.0);
  std::memcpy(xpad.data(), x, sizeof(double) * (size_t)n * d);
}

// X_F = trim(IDWT(f (.) DWT(pad(X)))): Sec. 3.1 steps 3, 5, 6.
// If coeffs_out != nullptr the unfiltered coefficients are returned too.
void haar_filter(const double* x, int n, int d, int L, const double* f, double* xf,
                 std::vector<vec>* coeffs_out) {
  int npad = next_pow2(n);
  vec xpad;
  pad_rows(x, n, d, npad, xpad);
  std::vector<vec> coeffs;
  haar_dwt(xpad, npad, d, L, coeffs);
  if (coeffs_out) *coeffs_out = coeffs;
  for (int i = 0; i <= L; ++i)
    for (size_t j = 0; j < coeffs[i].size(); ++j) coeffs[i][j] *= f[i];
  vec rec;
  haar_idwt(coeffs, npad, d, L, rec);
  std::memcpy(xf, rec.data(), sizeof(double) * (size_t)n * d);  // trim to orig_len
}

double sigmoid(double u) { return 1.0 / (1.0 + std::exp(-u)); }

struct Cfg {
  int B, H, n, d, L, m;
  double eps, bw_floor;
  int gate_per_head;
};

// Eq. 1: qbar[b][h][c] = mean over the n real rows of Q.
void mean_pool(const Cfg& g, const double* Q, vec& qbar) {
  qbar.assign((size_t)g.B * g.H * g.d, 0.0);
  for (int s = 0; s < g.B * g.H; ++s) {
    const double* q = Q + (size_t)s * g.n * g.d;
    for (int c = 0; c < g.d; ++c) {
      double acc = 0.0;
      for (int t = 0; t < g.n; ++t) acc += q[(size_t)t * g.d + c];
      qbar[(size_t)s * g.d + c] = acc / g.n;
    }
  }
}

// Eqs. 2-3.  g is one linear layer (Algorithm 1's W_filter) plus a bias:
//   per-head gate (Sec. 3.1):  u[b][h] = gate_w[h]^T qbar[b][h] + gate_b[h]
//   batch-wide gate (Alg. 1):  u[b]    = sum_h gate_w[h]^T qbar[b][h] + gate_b[0]
// f = sigmoid(u) * omega.  u, sg (= sigmoid(u)) and f are (B, H, L+1).
void gate(const Cfg& g, const vec& qbar, const double* gate_w, const double* gate_b,
          const double* omega, vec& u, vec& sg, vec& f) {
  int L1 = g.L + 1;
  u.assign((size_t)g.B * g.H * L1, 0.0);
  for (int b = 0; b < g.B; ++b) {
    for (int h = 0; h < g.H; ++h)
      for (int i = 0; i < L1; ++i) {
        double acc = 0.0;
        if (gate_w)
          for (int c = 0; c < g.d; ++c)
            acc += (double)gate_w[((size_t)h * g.d + c) * L1 + i] *
                   qbar[((size_t)b * g.H + h) * g.d + c];
        u[((size_t)b * g.H + h) * L1 + i] = acc;
      }
    if (!g.gate_per_head) {
      for (int i = 0; i < L1; ++i) {
        double tot = 0.0;
        for (int h = 0; h < g.H; ++h) tot += u[((size_t)b * g.H + h) * L1 + i];
        for (int h = 0; h < g.H; ++h) u[((size_t)b * g.H + h) * L1 + i] = tot;
      }
    }
    for (int h = 0; h < g.H; ++h)
      for (int i = 0; i < L1; ++i) {
        int hb = g.gate_per_head ? h : 0;
        if (gate_b) u[((size_t)b * g.H + h) * L1 + i] += (double)gate_b[(size_t)hb * L1 + i];
      }
  }
  sg.resize(u.size());
  f.resize(u.size());
  for (size_t j = 0; j < u.size(); ++j) {
    sg[j] = sigmoid(u[j]);
    f[j] = sg[j] * (double)omega[j % L1];
  }
}

// Eq. 6 with Algorithm 1's scalings: a = x W / bw, phi = max(0, a) / sqrt(m), one row.
inline void feature_row(const double* x, const vec& W, int d, int m, double bw, double* a,
                        double* phi) {
  for (int r = 0; r < m; ++r) a[r] = 0.0;
  for (int c = 0; c < d; ++c) {
    double xc = x[c];
    const double* w = &W[(size_t)c * m];
    for (int r = 0; r < m; ++r) a[r] += xc * w[r];
  }
  double inv_sqrt_m = 1.0 / std::sqrt((double)m);
  for (int r = 0; r < m; ++r) {
    a[r] /= bw;
    phi[r] = (a[r] > 0.0 ? a[r] : 0.0) * inv_sqrt_m;
  }
}

void to_double(const double* src, size_t count, vec& dst) {
  dst.resize(count);
  for (size_t i = 0; i < count; ++i) dst[i] = (double)src[i];
}

}  // namespace

extern "C" {

// ---- building blocks exported for the pin tests ---------------------------------------------

// Literal analysis of an (n x d) signal; n is zero-padded to npad = next_pow2(n).
// coeffs_flat receives [d_1 | d_2 | ... | d_L | a_L] back to back (npad*d doubles).
int wersa_oracle_dwt(const double* x, int n, int d, int L, double* coeffs_flat) {
  int npad = next_pow2(n);
  if (L < 1 || (npad >> L) < 1) return 1;
  vec xpad;
  pad_rows(x, n, d, npad, xpad);
  std::vector<vec> coeffs;
  haar_dwt(xpad, npad, d, L, coeffs);
  size_t off = 0;
  for (int i = 0; i <= L; ++i) {
    std::memcpy(coeffs_flat + off, coeffs[i].data(), sizeof(double) * coeffs[i].size());
    off += coeffs[i].size();
  }
  return 0;
}

// Literal synthesis from the flat coefficient list; writes npad rows.
int wersa_oracle_idwt(const double* coeffs_flat, int npad, int d, int L, double* x) {
  if (L < 1 || (npad >> L) < 1 || next_pow2(npad) != npad) return 1;
  std::vector<vec> coeffs(L + 1);
  size_t off = 0;
  for (int i = 0; i <= L; ++i) {
    size_t rows = (i < L) ? (size_t)(npad >> (i + 1)) : (size_t)(npad >> L);
    coeffs[i].assign(coeffs_flat + off, coeffs_flat + off + rows * d);
    off += rows * d;
  }
  vec out;
  haar_idwt(coeffs, npad, d, L, out);
  std::memcpy(x, out.data(), sizeof(double) * (size_t)npad * d);
  return 0;
}

// Pad, analyse, scale band i by f[i] (i = 0..L: d_1..d_L, a_L), synthesise, trim.
int wersa_oracle_filter(const double* x, int n, int d, int L, const double* f, double* xf) {
  if (L < 1 || (next_pow2(n) >> L) < 1) return 1;
  haar_filter(x, n, d, L, f, xf, nullptr);
  return 0;
}

// phi(x) for rows of x (n x d), W (d x m) row-major.
int wersa_oracle_features(const double* x, int n, int d, int m, const double* W, double beta,
                          double bw_floor, double* phi) {
  double bw = beta > bw_floor ? beta : bw_floor;
  vec Wv(W, W + (size_t)d * m), a(m);
  for (int t = 0; t < n; ++t)
    feature_row(x + (size_t)t * d, Wv, d, m, bw, a.data(), phi + (size_t)t * m);
  return 0;
}

// Gate only: qbar (B,H,d), f (B,H,L+1).
int wersa_oracle_gate(int B, int H, int n, int d, int L, int gate_per_head, const double* Q,
                      const double* gate_w, const double* gate_b, const double* omega,
                      double* qbar_out, double* f_out) {
  Cfg g{B, H, n, d, L, 0, 0.0, 0.0, gate_per_head};
  vec qbar, u, sg, f;
  mean_pool(g, Q, qbar);
  gate(g, qbar, gate_w, gate_b, omega, u, sg, f);
  if (qbar_out) std::memcpy(qbar_out, qbar.data(), sizeof(double) * qbar.size());
  if (f_out) std::memcpy(f_out, f.data(), sizeof(double) * f.size());
  return 0;
}

// ---- whole forward --------------------------------------------------------------------------
//
// Q, K, V: (B,H,n,d) row-major doubles (the exact values the GPU receives, widened exactly
// from fp32 / bf16 by the caller).  W: (d,m).  gate_w: (H,d,L+1) or NULL (= 0).  gate_b: (H,L+1) or NULL.
// omega: (L+1).  Outputs (any may be NULL): O (B,H,n,d), f (B,H,L+1), qbar (B,H,d),
// S (B,H,m,d), z (B,H,m), D (B,H,n).
// sample_rows/n_sample: if n_sample > 0 only these query rows of every slab get an output
// (the rest of O and D is left untouched); the key side always runs over all n rows.
int wersa_oracle_forward(int B, int H, int n, int d, int L, int m, double eps, double bw_floor,
                         int gate_per_head, const double* Q, const double* K, const double* V,
                         const double* W, double beta, const double* gate_w, const double* gate_b,
                         const double* omega, double* O, double* f_out, double* qbar_out,
                         double* S_out, double* z_out, double* D_out, const int* sample_rows,
                         int n_sample) {
  if (B < 1 || H < 1 || n < 1 || d < 1 || m < 1 || L < 1 || (next_pow2(n) >> L) < 1) return 1;
  Cfg g{B, H, n, d, L, m, eps, bw_floor, gate_per_head};
  int L1 = L + 1;
  vec qbar, u, sg, f;
  mean_pool(g, Q, qbar);                            // Eq. 1
  gate(g, qbar, gate_w, gate_b, omega, u, sg, f);   // Eqs. 2-3
  if (qbar_out) std::memcpy(qbar_out, qbar.data(), sizeof(double) * qbar.size());
  if (f_out) std::memcpy(f_out, f.data(), sizeof(double) * f.size());
  vec Wd;
  to_double(W, (size_t)d * m, Wd);
  double bw = beta > bw_floor ? beta : bw_floor;    // Algorithm 1: bw = max(beta, floor)

#pragma omp parallel for schedule(dynamic, 1)
  for (int s = 0; s < B * H; ++s) {
    size_t base = (size_t)s * n * d;
    vec q, k, v, qf((size_t)n * d), kf((size_t)n * d);
    to_double(Q + base, (size_t)n * d, q);
    to_double(K + base, (size_t)n * d, k);
    to_double(V + base, (size_t)n * d, v);
    const double* fs = &f[(size_t)s * L1];
    haar_filter(q.data(), n, d, L, fs, qf.data(), nullptr);   // steps 3, 5, 6
    haar_filter(k.data(), n, d, L, fs, kf.data(), nullptr);
    // Key summary, Eq. 7: S = phi(K_F)^T V, z = phi(K_F)^T 1.
    vec S((size_t)m * d, 0.0), z(m, 0.0), a(m), phi(m);
    for (int t = 0; t < n; ++t) {
      feature_row(&kf[(size_t)t * d], Wd, d, m, bw, a.data(), phi.data());
      const double* vt = &v[(size_t)t * d];
      for (int r = 0; r < m; ++r) {
        double p = phi[r];
        z[r] += p;
        double* Sr = &S[(size_t)r * d];
        for (int c = 0; c < d; ++c) Sr[c] += p * vt[c];
      }
    }
    if (S_out) std::memcpy(S_out + (size_t)s * m * d, S.data(), sizeof(double) * S.size());
    if (z_out) std::memcpy(z_out + (size_t)s * m, z.data(), sizeof(double) * z.size());
    // Output, Eq. 7: O = phi(Q_F) S / (phi(Q_F) z + eps).
    int rows = n_sample > 0 ? n_sample : n;
    vec num(d);
    for (int j = 0; j < rows; ++j) {
      int t = n_sample > 0 ? sample_rows[j] : j;
      if (t < 0 || t >= n) continue;
      feature_row(&qf[(size_t)t * d], Wd, d, m, bw, a.data(), phi.data());
      for (int c = 0; c < d; ++c) num[c] = 0.0;
      double den = 0.0;
      for (int r = 0; r < m; ++r) {
        double p = phi[r];
        den += p * z[r];
        const double* Sr = &S[(size_t)r * d];
        for (int c = 0; c < d; ++c) num[c] += p * Sr[c];
      }
      den += eps;
      if (D_out) D_out[(size_t)s * n + t] = den;
      if (O)
        for (int c = 0; c < d; ++c) O[base + (size_t)t * d + c] = num[c] / den;
    }
  }
  return 0;
}

// ---- whole backward -------------------------------------------------------------------------
//
// Chain rule through the forward steps in reverse.  dO: (B,H,n,d) doubles.
// Outputs: dQ, dK, dV (B,H,n,d); dbeta (1); dgate_w (H,d,L+1); dgate_b (H,L+1); domega (L+1).
// dbeta_closed (optional, 1): the closed form 2*eps/bw * sum dD that positive homogeneity
// of ReLU implies; the test-suite asserts that it equals the generic chain-rule value.
int wersa_oracle_backward(int B, int H, int n, int d, int L, int m, double eps, double bw_floor,
                          int gate_per_head, const double* Q, const double* K, const double* V,
                          const double* W, double beta, const double* gate_w,
                          const double* gate_b, const double* omega, const double* dO, double* dQ,
                          double* dK, double* dV, double* dbeta, double* dgate_w,
                          double* dgate_b, double* domega, double* dbeta_closed) {
  if (B < 1 || H < 1 || n < 1 || d < 1 || m < 1 || L < 1 || (next_pow2(n) >> L) < 1) return 1;
  Cfg g{B, H, n, d, L, m, eps, bw_floor, gate_per_head};
  int L1 = L + 1;
  int npad = next_pow2(n);
  vec qbar, u, sg, f;
  mean_pool(g, Q, qbar);
  gate(g, qbar, gate_w, gate_b, omega, u, sg, f);
  vec Wd;
  to_double(W, (size_t)d * m, Wd);
  double bw = beta > bw_floor ? beta : bw_floor;
  double inv_sqrt_m = 1.0 / std::sqrt((double)m);

  vec df_all((size_t)B * H * L1, 0.0);
  std::vector<long double> dbw_slab(B * H, 0.0L), sum_dD_slab(B * H, 0.0L);

#pragma omp parallel for schedule(dynamic, 1)
  for (int s = 0; s < B * H; ++s) {
    size_t base = (size_t)s * n * d;
    vec q, k, v, go, qf((size_t)n * d), kf((size_t)n * d);
    to_double(Q + base, (size_t)n * d, q);
    to_double(K + base, (size_t)n * d, k);
    to_double(V + base, (size_t)n * d, v);
    to_double(dO + base, (size_t)n * d, go);
    const double* fs = &f[(size_t)s * L1];
    std::vector<vec> qc, kc;  // unfiltered wavelet coefficients of Q and K
    haar_filter(q.data(), n, d, L, fs, qf.data(), &qc);
    haar_filter(k.data(), n, d, L, fs, kf.data(), &kc);

    // Forward quantities, kept whole (n x m) for clarity.
    vec Aq((size_t)n * m), Pq((size_t)n * m), Ak((size_t)n * m), Pk((size_t)n * m);
    for (int t = 0; t < n; ++t) {
      feature_row(&qf[(size_t)t * d], Wd, d, m, bw, &Aq[(size_t)t * m], &Pq[(size_t)t * m]);
      feature_row(&kf[(size_t)t * d], Wd, d, m, bw, &Ak[(size_t)t * m], &Pk[(size_t)t * m]);
    }
    vec S((size_t)m * d, 0.0), z(m, 0.0);
    for (int t = 0; t < n; ++t)
      for (int r = 0; r < m; ++r) {
        double p = Pk[(size_t)t * m + r];
        z[r] += p;
        for (int c = 0; c < d; ++c) S[(size_t)r * d + c] += p * v[(size_t)t * d + c];
      }
    vec N((size_t)n * d, 0.0), D(n, 0.0), Oo((size_t)n * d);
    for (int t = 0; t < n; ++t) {
      double den = 0.0;
      for (int r = 0; r < m; ++r) {
        double p = Pq[(size_t)t * m + r];
        den += p * z[r];
        for (int c = 0; c < d; ++c) N[(size_t)t * d + c] += p * S[(size_t)r * d + c];
      }
      D[t] = den + eps;
      for (int c = 0; c < d; ++c) Oo[(size_t)t * d + c] = N[(size_t)t * d + c] / D[t];
    }

    // O = N / D.
    vec dN((size_t)n * d), dD(n, 0.0);
    long double sum_dD = 0.0L;
    for (int t = 0; t < n; ++t) {
      double acc = 0.0;
      for (int c = 0; c < d; ++c) {
        dN[(size_t)t * d + c] = go[(size_t)t * d + c] / D[t];
        acc += go[(size_t)t * d + c] * Oo[(size_t)t * d + c];
      }
      dD[t] = -acc / D[t];
      sum_dD += dD[t];
    }
    sum_dD_slab[s] = sum_dD;
    // N = Pq S, D = Pq z + eps.
    vec dPq((size_t)n * m, 0.0), dS((size_t)m * d, 0.0), dz(m, 0.0);
    for (int t = 0; t < n; ++t)
      for (int r = 0; r < m; ++r) {
        double p = Pq[(size_t)t * m + r], acc = dD[t] * z[r];
        for (int c = 0; c < d; ++c) {
          acc += dN[(size_t)t * d + c] * S[(size_t)r * d + c];
          dS[(size_t)r * d + c] += p * dN[(size_t)t * d + c];
        }
        dPq[(size_t)t * m + r] = acc;
        dz[r] += p * dD[t];
      }
    // S = Pk^T V, z = Pk^T 1.
    vec dPk((size_t)n * m), dv((size_t)n * d, 0.0);
    for (int t = 0; t < n; ++t)
      for (int r = 0; r < m; ++r) {
        double p = Pk[(size_t)t * m + r], acc = dz[r];
        for (int c = 0; c < d; ++c) {
          acc += v[(size_t)t * d + c] * dS[(size_t)r * d + c];
          dv[(size_t)t * d + c] += p * dS[(size_t)r * d + c];
        }
        dPk[(size_t)t * m + r] = acc;
      }
    std::memcpy(dV + base, dv.data(), sizeof(double) * dv.size());
    // P = max(0, A)/sqrt(m);  A = X_F W / bw.
    vec dqf((size_t)n * d, 0.0), dkf((size_t)n * d, 0.0);
    long double dbw = 0.0L;
    for (int t = 0; t < n; ++t)
      for (int r = 0; r < m; ++r) {
        double aq = Aq[(size_t)t * m + r], ak = Ak[(size_t)t * m + r];
        double dAq = aq > 0.0 ? dPq[(size_t)t * m + r] * inv_sqrt_m : 0.0;
        double dAk = ak > 0.0 ? dPk[(size_t)t * m + r] * inv_sqrt_m : 0.0;
        dbw += -(long double)(dAq * aq) / bw;
        dbw += -(long double)(dAk * ak) / bw;
        for (int c = 0; c < d; ++c) {
          dqf[(size_t)t * d + c] += dAq * Wd[(size_t)c * m + r] / bw;
          dkf[(size_t)t * d + c] += dAk * Wd[(size_t)c * m + r] / bw;
        }
      }
    dbw_slab[s] = dbw;
    // X_F = trim(IDWT(f (.) DWT(pad X))).  Adjoint of trim = zero-pad, adjoint of the
    // orthonormal synthesis = analysis, adjoint of analysis = synthesis, adjoint of pad = trim.
    for (int which = 0; which < 2; ++which) {
      const vec& gxf = which == 0 ? dqf : dkf;
      const std::vector<vec>& xc = which == 0 ? qc : kc;
      vec gpad;
      pad_rows(gxf.data(), n, d, npad, gpad);
      std::vector<vec> gc;
      haar_dwt(gpad, npad, d, L, gc);
      for (int i = 0; i <= L; ++i) {
        double acc = 0.0;
        for (size_t j = 0; j < gc[i].size(); ++j) {
          acc += gc[i][j] * xc[i][j];   // d/df_i of (f_i * coeff)
          gc[i][j] *= fs[i];            // d/dcoeff
        }
        df_all[(size_t)s * L1 + i] += acc;
      }
      vec gx;
      haar_idwt(gc, npad, d, L, gx);
      double* dst = (which == 0 ? dQ : dK) + base;
      std::memcpy(dst, gx.data(), sizeof(double) * (size_t)n * d);
    }
  }

  // bw = max(beta, floor).
  long double dbw_tot = 0.0L, sum_dD_tot = 0.0L;
  for (int s = 0; s < B * H; ++s) {
    dbw_tot += dbw_slab[s];
    sum_dD_tot += sum_dD_slab[s];
  }
  bool live = beta > bw_floor;
  if (dbeta) *dbeta = live ? (double)dbw_tot : 0.0;
  if (dbeta_closed) *dbeta_closed = live ? (double)(2.0L * eps / bw * sum_dD_tot) : 0.0;

  // f = sigmoid(u) * omega; u = gate(qbar); qbar = mean(Q).
  vec gw((size_t)H * d * L1, 0.0), gb((size_t)H * L1, 0.0), gom(L1, 0.0);
  for (int b = 0; b < B; ++b) {
    vec df((size_t)H * L1);
    for (int h = 0; h < H; ++h)
      for (int i = 0; i < L1; ++i) df[(size_t)h * L1 + i] = df_all[((size_t)b * H + h) * L1 + i];
    if (!gate_per_head) {  // one f shared by all heads of the batch element
      for (int i = 0; i < L1; ++i) {
        double tot = 0.0;
        for (int h = 0; h < H; ++h) tot += df[(size_t)h * L1 + i];
        df[i] = tot;
      }
    }
    int groups = gate_per_head ? H : 1;
    for (int gi = 0; gi < groups; ++gi) {
      vec du(L1);
      for (int i = 0; i < L1; ++i) {
        double sgi = sg[((size_t)b * H + gi) * L1 + i];
        double dfi = df[(size_t)gi * L1 + i];
        gom[i] += dfi * sgi;
        du[i] = dfi * (double)omega[i] * sgi * (1.0 - sgi);
        gb[(size_t)gi * L1 + i] += du[i];
      }
      int h0 = gate_per_head ? gi : 0, h1 = gate_per_head ? gi + 1 : H;
      for (int h = h0; h < h1; ++h) {
        int s = b * H + h;
        for (int c = 0; c < d; ++c) {
          double dq = 0.0;
          for (int i = 0; i < L1; ++i) {
            gw[((size_t)h * d + c) * L1 + i] += qbar[(size_t)s * d + c] * du[i];
            if (gate_w) dq += (double)gate_w[((size_t)h * d + c) * L1 + i] * du[i];
          }
          for (int t = 0; t < n; ++t) dQ[(size_t)s * n * d + (size_t)t * d + c] += dq / n;
        }
      }
    }
  }
  if (dgate_w) std::memcpy(dgate_w, gw.data(), sizeof(double) * gw.size());
  if (dgate_b) std::memcpy(dgate_b, gb.data(), sizeof(double) * gb.size());
  if (domega) std::memcpy(domega, gom.data(), sizeof(double) * gom.size());
  return 0;
}

int wersa_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"

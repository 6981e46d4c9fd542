/*
 * fp64 CPU oracle for token-wise adaptive low-rank KV-cache compression.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow definition of what
 * the CUDA library computes.  It shares no code with the CUDA path, is never
 * linked into the product library, and must only be called from tests, the
 * smoke check and the benchmark's CPU-baseline leg.
 *
 * Every function follows one passage of the paper:
 *   oracle_project       Eq. 1  (x~ = x U, projection to the spectral space)
 *   oracle_gate_logits   Eq. 5  (z = x~ W + b, the argument of the softmax)
 *   oracle_gate_rank     Eq. 5, Eq. 6, Eq. 8  (softmax, cumsum, Flip, threshold)
 *   oracle_reconstruct   Eq. 2 + Eq. 3  (hard prefix mask, dynamic low-rank reconstruction)
 *   oracle_rope          Sec. 3.2, text after Eq. 3 (RoPE on reconstructed keys)
 *   oracle_decode_attn   Eq. 3 + reshape to heads + RoPE + softmax attention
 *
 * Conventions the paper leaves open are the ones the library documents:
 *   - Flip is a literal index reversal: m_i = c_{d+1-i} (1-based).
 *   - The hard mask uses a strict comparison m_i > tau.
 *   - RoPE pairs element i with i + d_h/2 ("rotate half"), angle pos * base^(-2i/d_h).
 *   - Attention scale is passed in (1/sqrt(d_h) by default), no masking: the
 *     single decode query attends to every cached token of its sequence.
 *
 * No blocking, fusion or reordering: loops are written in the order of the
 * formulas so they can be checked against the paper by eye.  OpenMP is used
 * only over independent tokens / heads.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 1: x~[t, :] = x[t, :] U.   U is [d x d] row-major: row j holds the weights of input
 * dimension j, column n is the n-th axis of the spectral space. */
void oracle_project(const double* x, const double* U, int64_t n_tok, int d, double* xt) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < n_tok; ++t) {
    double* o = xt + t * d;
    for (int n = 0; n < d; ++n) {
      double acc = 0.0;
      for (int j = 0; j < d; ++j) acc += x[t * d + j] * U[(int64_t)j * d + n];
      o[n] = acc;
    }
  }
}

/* Eq. 5 (inside the softmax): z[t, :] = x~[t, :] W + b.   W is [d x d] row-major. */
void oracle_gate_logits(const double* xt, const double* W, const double* b,
                        int64_t n_tok, int d, double* z) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < n_tok; ++t) {
    const double* x = xt + t * d;
    double* zt = z + t * d;
    for (int n = 0; n < d; ++n) zt[n] = b ? b[n] : 0.0;
    for (int j = 0; j < d; ++j) {
      const double xj = x[j];
      const double* Wj = W + (int64_t)j * d;
      for (int n = 0; n < d; ++n) zt[n] += xj * Wj[n];
    }
  }
}

/*
 * Eq. 5: p = Softmax(z);  Eq. 6: m = Flip(cumsum(p));  Eq. 8: m_hard_i = 1[m_i > tau].
 * The retained rank is r = sum_i m_hard_i (the numerator of Eq. 4).
 * Outputs per token: r, margin = min_n |c_n - tau| / tau (distance of the
 * closest cumulative sum from the threshold; used by tests to reject inputs
 * whose integer result could depend on rounding), and optionally the soft mask.
 */
void oracle_gate_rank(const double* z, int64_t n_tok, int d, double tau,
                      int32_t* r_out, double* margin_out, double* m_soft) {
#pragma omp parallel
  {
    double* p = (double*)malloc(sizeof(double) * d);
    double* c = (double*)malloc(sizeof(double) * d);
    double* m = (double*)malloc(sizeof(double) * d);
#pragma omp for schedule(static)
    for (int64_t t = 0; t < n_tok; ++t) {
      const double* zt = z + t * d;
      /* softmax */
      double zmax = zt[0];
      for (int j = 1; j < d; ++j) if (zt[j] > zmax) zmax = zt[j];
      double sum = 0.0;
      for (int j = 0; j < d; ++j) { p[j] = exp(zt[j] - zmax); sum += p[j]; }
      for (int j = 0; j < d; ++j) p[j] /= sum;
      /* cumsum */
      double run = 0.0;
      for (int n = 0; n < d; ++n) { run += p[n]; c[n] = run; }
      /* Flip: m_i = c_{d+1-i}, 1-based  ->  m[i] = c[d-1-i], 0-based */
      for (int i = 0; i < d; ++i) m[i] = c[d - 1 - i];
      /* hard mask and rank */
      int32_t r = 0;
      for (int i = 0; i < d; ++i) if (m[i] > tau) r += 1;
      r_out[t] = r;
      if (margin_out) {
        double best = INFINITY;
        for (int n = 0; n < d; ++n) {
          double g = fabs(c[n] - tau) / tau;
          if (g < best) best = g;
        }
        margin_out[t] = best;
      }
      if (m_soft) memcpy(m_soft + t * d, m, sizeof(double) * d);
    }
    free(p); free(c); free(m);
  }
}

/*
 * Eq. 2 + Eq. 3: xhat = x~ (.) m_hard with m_hard a prefix of r ones; the
 * retained index set is I = {0..r-1}; xbar = xhat[I] Uinv[I, :].
 * xt: [n_tok x d], r: [n_tok], Uinv: [d x d] row-major (row j = spectral index j).
 */
void oracle_reconstruct(const double* xt, const int32_t* r, const double* Uinv,
                        int64_t n_tok, int d, double* xbar) {
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < n_tok; ++t) {
    double* o = xbar + t * d;
    for (int n = 0; n < d; ++n) o[n] = 0.0;
    for (int j = 0; j < r[t]; ++j) {
      const double xj = xt[t * d + j];
      const double* Uj = Uinv + (int64_t)j * d;
      for (int n = 0; n < d; ++n) o[n] += xj * Uj[n];
    }
  }
}

/*
 * RoPE on multi-head keys (text after Eq. 3).  k: [n_tok x n_heads x d_h], in place.
 * Pair (i, i + d_h/2) of every head is rotated by angle pos[t] * base^(-2i/d_h).
 */
void oracle_rope(double* k, const int32_t* pos, int64_t n_tok, int n_heads, int d_h,
                 double base) {
  const int half = d_h / 2;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < n_tok; ++t) {
    for (int i = 0; i < half; ++i) {
      const double theta = pow(base, -2.0 * (double)i / (double)d_h);
      const double ang = (double)pos[t] * theta;
      const double cs = cos(ang), sn = sin(ang);
      for (int g = 0; g < n_heads; ++g) {
        double* kg = k + (t * n_heads + g) * d_h;
        const double a = kg[i], b = kg[i + half];
        kg[i] = a * cs - b * sn;
        kg[i + half] = b * cs + a * sn;
      }
    }
  }
}

/*
 * One decode-attention step for ONE sequence (Eq. 3, reshape, RoPE, attention).
 *   xk, xv : [T x d_kv] spectral states as cached (only the first rk[t] / rv[t]
 *            entries of a row are ever read: the rest was discarded, Eq. 2)
 *   pos    : [T] positions, q : [Hq x d_h] (already rotated at its own position)
 *   out    : [Hq x d_h]
 * Query head h reads KV head g = h / (Hq / Hkv).  Softmax is the two-pass
 * textbook form over all T tokens.  Returns 0, or -1 if memory ran out.
 */
int oracle_decode_attn(const double* xk, const double* xv, const int32_t* rk,
                       const int32_t* rv, const int32_t* pos, int64_t T,
                       const double* Uinv_k, const double* Uinv_v, const double* q,
                       int Hq, int Hkv, int d_h, double rope_base, double sm_scale,
                       double* out) {
  const int d = Hkv * d_h;
  const int rep = Hq / Hkv;
  double* kbar = (double*)malloc(sizeof(double) * (size_t)T * d);
  double* vbar = (double*)malloc(sizeof(double) * (size_t)T * d);
  if (!kbar || !vbar) { free(kbar); free(vbar); return -1; }
  oracle_reconstruct(xk, rk, Uinv_k, T, d, kbar);   /* Eq. 3 for keys   */
  oracle_reconstruct(xv, rv, Uinv_v, T, d, vbar);   /* Eq. 3 for values */
  oracle_rope(kbar, pos, T, Hkv, d_h, rope_base);   /* reshape + RoPE   */
#pragma omp parallel for schedule(static)
  for (int h = 0; h < Hq; ++h) {
    const int g = h / rep;
    const double* qh = q + (int64_t)h * d_h;
    double* s = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    double smax = -INFINITY;
    for (int64_t t = 0; t < T; ++t) {
      const double* kt = kbar + (t * Hkv + g) * d_h;
      double acc = 0.0;
      for (int i = 0; i < d_h; ++i) acc += qh[i] * kt[i];
      s[t] = acc * sm_scale;
      if (s[t] > smax) smax = s[t];
    }
    double denom = 0.0;
    for (int64_t t = 0; t < T; ++t) { s[t] = exp(s[t] - smax); denom += s[t]; }
    double* oh = out + (int64_t)h * d_h;
    for (int i = 0; i < d_h; ++i) oh[i] = 0.0;
    for (int64_t t = 0; t < T; ++t) {
      const double a = s[t] / denom;
      const double* vt = vbar + (t * Hkv + g) * d_h;
      for (int i = 0; i < d_h; ++i) oh[i] += a * vt[i];
    }
    free(s);
  }
  free(kbar); free(vbar);
  return 0;
}

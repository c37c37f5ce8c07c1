/*
 * fp64 CPU oracle for first-layer bidirectional RoPE attention with the
 * FACache / RoPECache partial-state formulation.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, obviously-correct
 * definition the CUDA path is checked against.  It shares no code, header,
 * table or constant with the CUDA path and must never be called from the
 * product path.
 *
 * What is written out here, and where the paper states it:
 *   - RoPE on Q and K only, V untouched (Sec. 3.3.2, Eq. 1).  Pairing is the
 *     half-split (c, c + d/2), frequency theta^(-2c/d), position = 0-based
 *     index of the token inside its own sequence.
 *   - Softmax attention without any mask, O = diag(l)^-1 O~ (Sec. 3.3.3 text
 *     after Eq. 6; App. B.2) and L = m + log l (Algorithm 1, output L_i).
 *   - The online-softmax recurrence (m, alpha, P~, l, O~) of Eq. 2-6, used to
 *     form a partial state over an arbitrary subset of keys, and the merge of
 *     two partial states that the same recurrence implies.
 *   - The reuse pass of Algorithm 1 (GenStep = False): fixed queries start
 *     from the cached state and visit only the current block's keys.
 *
 * All arrays are row-major double; token-major [T, H, d].
 * Parity pins (tests/test_oracle_*.py): brute force on tiny inputs, closed
 * forms (q = 0, equal values, one dominant key), torch SDPA with RoPE
 * disabled, RoPE isometry / shift invariance / Toeplitz structure, key
 * permutation invariance, split-merge identity on random partitions,
 * GQA == repeated MHA, packed == each sequence alone.  The paper prints no
 * numeric worked example, so there is no paper-value pin.
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

/* R(p) x for one vector (Eq. 1; half-split pairing). */
static void rope_vec(const double* x, int d, double p, double theta, double* y) {
  int half = d / 2;
  for (int c = 0; c < half; ++c) {
    double f = pow(theta, -2.0 * (double)c / (double)d);
    double a = p * f;
    double cs = cos(a), sn = sin(a);
    y[c] = x[c] * cs - x[c + half] * sn;
    y[c + half] = x[c + half] * cs + x[c] * sn;
  }
}

/* y[t,h,:] = R(pos[t]) x[t,h,:] for all tokens and heads. */
void oracle_rope(const double* x, const int32_t* pos, int T, int H, int d,
                 double theta, double* y) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t)
    for (int h = 0; h < H; ++h)
      rope_vec(x + ((size_t)t * H + h) * d, d, (double)pos[t], theta,
               y + ((size_t)t * H + h) * d);
}

static int seq_of_token(const int32_t* cu, int B, int t) {
  for (int b = 0; b < B; ++b)
    if (t >= cu[b] && t < cu[b + 1]) return b;
  return -1;
}

/*
 * The plain definition, no tiles, no state, no cache.
 * q [T,Hq,d], k,v [T,Hkv,d] are PRE-RoPE.  For every listed row i (a packed
 * token index) and every query head h:
 *    s_j = scale <R(p_i) q_i, R(p_j) k_j>,  j over all tokens of i's sequence
 *    out = sum_j softmax(s)_j v_j,  lse = max + log sum exp(s - max)
 * out [n_rows,Hq,d], lse [n_rows,Hq].  kv head of query head h is h / (Hq/Hkv).
 */
void oracle_attention(const double* q, const double* k, const double* v,
                      const int32_t* cu, int B, int Hq, int Hkv, int d,
                      double theta, double scale, const int32_t* rows,
                      int n_rows, double* out, double* lse) {
  int T = cu[B];
  int g = Hq / Hkv;
  /* rotate every key once; this is the same R(p) applied per token */
  double* kr = (double*)malloc((size_t)T * Hkv * d * sizeof(double));
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    int b = seq_of_token(cu, B, t);
    for (int h = 0; h < Hkv; ++h)
      rope_vec(k + ((size_t)t * Hkv + h) * d, d, (double)(t - cu[b]), theta,
               kr + ((size_t)t * Hkv + h) * d);
  }
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
  for (int r = 0; r < n_rows; ++r) {
    for (int h = 0; h < Hq; ++h) {
      int i = rows[r];
      int b = seq_of_token(cu, B, i);
      int lo = cu[b], hi = cu[b + 1], n = hi - lo;
      int kh = h / g;
      double* qr = (double*)malloc((size_t)d * sizeof(double));
      double* s = (double*)malloc((size_t)n * sizeof(double));
      rope_vec(q + ((size_t)i * Hq + h) * d, d, (double)(i - lo), theta, qr);
      double M = -INFINITY;
      for (int j = 0; j < n; ++j) {
        const double* kj = kr + ((size_t)(lo + j) * Hkv + kh) * d;
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += qr[c] * kj[c];
        s[j] = scale * acc;
        if (s[j] > M) M = s[j];
      }
      double Z = 0.0;
      for (int j = 0; j < n; ++j) Z += exp(s[j] - M);
      double* o = out + ((size_t)r * Hq + h) * d;
      for (int c = 0; c < d; ++c) o[c] = 0.0;
      for (int j = 0; j < n; ++j) {
        double w = exp(s[j] - M) / Z;
        const double* vj = v + ((size_t)(lo + j) * Hkv + kh) * d;
        for (int c = 0; c < d; ++c) o[c] += w * vj[c];
      }
      lse[(size_t)r * Hq + h] = M + log(Z);
      free(qr);
      free(s);
    }
  }
  free(kr);
}

/*
 * Partial online-softmax state of ONE query vector over a subset of keys,
 * streamed in column tiles of Bc keys exactly as Eq. 2-6 state it:
 *   m_j = max(m_{j-1}, rowmax(S_j)); alpha = exp(m_{j-1} - m_j);
 *   P~ = exp(S_j - m_j); l_j = alpha l_{j-1} + rowsum(P~);
 *   O~_j = alpha O~_{j-1} + P~ V_j.
 * qrot [d], krot [n,d] are ALREADY rotated, v [n,d]; keep[j] != 0 selects
 * key j.  A tile with no selected key leaves the state untouched.  Starts
 * from the state passed in (m, l, O); pass (-inf, 0, 0) for an empty state.
 */
void oracle_state_stream(const double* qrot, const double* krot,
                         const double* v, const uint8_t* keep, int n, int d,
                         double scale, int Bc, double* m, double* l,
                         double* O) {
  double* s = (double*)malloc((size_t)Bc * sizeof(double));
  for (int j0 = 0; j0 < n; j0 += Bc) {
    int j1 = j0 + Bc < n ? j0 + Bc : n;
    double rm = -INFINITY;
    for (int j = j0; j < j1; ++j) {
      if (!keep[j]) continue;
      double acc = 0.0;
      for (int c = 0; c < d; ++c) acc += qrot[c] * krot[(size_t)j * d + c];
      s[j - j0] = scale * acc;
      if (s[j - j0] > rm) rm = s[j - j0];
    }
    if (rm == -INFINITY) continue;
    double m_new = *m > rm ? *m : rm;
    double alpha = (*m == -INFINITY) ? 0.0 : exp(*m - m_new);
    double rs = 0.0;
    for (int c = 0; c < d; ++c) O[c] *= alpha;
    for (int j = j0; j < j1; ++j) {
      if (!keep[j]) continue;
      double p = exp(s[j - j0] - m_new);
      rs += p;
      for (int c = 0; c < d; ++c) O[c] += p * v[(size_t)j * d + c];
    }
    *l = alpha * (*l) + rs;
    *m = m_new;
  }
  free(s);
}

/* Merge of two partial states over disjoint key sets (Eq. 2-6 with the second
 * state playing the role of one more streamed tile).  Result in (m1,l1,O1). */
void oracle_state_merge(double* m1, double* l1, double* O1, double m2,
                        double l2, const double* O2, int d) {
  if (m2 == -INFINITY) return;
  double m = *m1 > m2 ? *m1 : m2;
  double a1 = (*m1 == -INFINITY) ? 0.0 : exp(*m1 - m);
  double a2 = exp(m2 - m);
  for (int c = 0; c < d; ++c) O1[c] = a1 * O1[c] + a2 * O2[c];
  *l1 = a1 * (*l1) + a2 * l2;
  *m1 = m;
}

/*
 * FACache build (Algorithm 1, GenStep = True, cache side): for every token i
 * and query head h, the state over the FIXED keys of i's sequence, i.e. all
 * keys whose is_block flag is 0.  q,k,v pre-RoPE, token-major.  Outputs
 * m,l [T,Hq], O [T,Hq,d].  Rows that are themselves block tokens get the same
 * treatment (their state is simply never used).
 */
void oracle_build_state(const double* q, const double* k, const double* v,
                        const int32_t* cu, int B, const uint8_t* is_block,
                        int Hq, int Hkv, int d, double theta, double scale,
                        int Bc, double* m, double* l, double* O) {
  int T = cu[B];
  int g = Hq / Hkv;
  int32_t* pos = (int32_t*)malloc((size_t)T * sizeof(int32_t));
  for (int t = 0; t < T; ++t) pos[t] = t - cu[seq_of_token(cu, B, t)];
  double* qr = (double*)malloc((size_t)T * Hq * d * sizeof(double));
  double* kr = (double*)malloc((size_t)T * Hkv * d * sizeof(double));
  oracle_rope(q, pos, T, Hq, d, theta, qr);
  oracle_rope(k, pos, T, Hkv, d, theta, kr);
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
  for (int i = 0; i < T; ++i) {
    for (int h = 0; h < Hq; ++h) {
      int b = seq_of_token(cu, B, i);
      int lo = cu[b], n = cu[b + 1] - lo, kh = h / g;
      double* kk = (double*)malloc((size_t)n * d * sizeof(double));
      double* vv = (double*)malloc((size_t)n * d * sizeof(double));
      uint8_t* keep = (uint8_t*)malloc((size_t)n);
      for (int j = 0; j < n; ++j) {
        memcpy(kk + (size_t)j * d, kr + ((size_t)(lo + j) * Hkv + kh) * d,
               d * sizeof(double));
        memcpy(vv + (size_t)j * d, v + ((size_t)(lo + j) * Hkv + kh) * d,
               d * sizeof(double));
        keep[j] = is_block[lo + j] ? 0 : 1;
      }
      double mm = -INFINITY, ll = 0.0;
      double* oo = O + ((size_t)i * Hq + h) * d;
      for (int c = 0; c < d; ++c) oo[c] = 0.0;
      oracle_state_stream(qr + ((size_t)i * Hq + h) * d, kk, vv, keep, n, d,
                          scale, Bc, &mm, &ll, oo);
      m[(size_t)i * Hq + h] = mm;
      l[(size_t)i * Hq + h] = ll;
      free(kk);
      free(vv);
      free(keep);
    }
  }
  free(pos);
  free(qr);
  free(kr);
}

/*
 * Reuse pass (Algorithm 1, GenStep = False) in fp64.  q,k,v are the CURRENT
 * pre-RoPE arrays (block rows hold this step's fresh values).  Fixed queries
 * start from the cached (m,l,O) and stream only block keys; block queries
 * start empty and stream all keys.  out [T,Hq,d], lse [T,Hq].
 */
void oracle_reuse_step(const double* q, const double* k, const double* v,
                       const int32_t* cu, int B, const uint8_t* is_block,
                       int Hq, int Hkv, int d, double theta, double scale,
                       int Bc, const double* mc, const double* lc,
                       const double* Oc, double* out, double* lse) {
  int T = cu[B];
  int g = Hq / Hkv;
  int32_t* pos = (int32_t*)malloc((size_t)T * sizeof(int32_t));
  for (int t = 0; t < T; ++t) pos[t] = t - cu[seq_of_token(cu, B, t)];
  double* qr = (double*)malloc((size_t)T * Hq * d * sizeof(double));
  double* kr = (double*)malloc((size_t)T * Hkv * d * sizeof(double));
  oracle_rope(q, pos, T, Hq, d, theta, qr);
  oracle_rope(k, pos, T, Hkv, d, theta, kr);
#pragma omp parallel for collapse(2) schedule(dynamic, 4)
  for (int i = 0; i < T; ++i) {
    for (int h = 0; h < Hq; ++h) {
      int b = seq_of_token(cu, B, i);
      int lo = cu[b], n = cu[b + 1] - lo, kh = h / g;
      double* kk = (double*)malloc((size_t)n * d * sizeof(double));
      double* vv = (double*)malloc((size_t)n * d * sizeof(double));
      uint8_t* keep = (uint8_t*)malloc((size_t)n);
      int fixed_q = !is_block[i];
      for (int j = 0; j < n; ++j) {
        memcpy(kk + (size_t)j * d, kr + ((size_t)(lo + j) * Hkv + kh) * d,
               d * sizeof(double));
        memcpy(vv + (size_t)j * d, v + ((size_t)(lo + j) * Hkv + kh) * d,
               d * sizeof(double));
        /* fixed query: only keys overlapping the block; block query: all */
        keep[j] = fixed_q ? (is_block[lo + j] ? 1 : 0) : 1;
      }
      double mm = -INFINITY, ll = 0.0;
      double* oo = out + ((size_t)i * Hq + h) * d;
      if (fixed_q) {
        mm = mc[(size_t)i * Hq + h];
        ll = lc[(size_t)i * Hq + h];
        memcpy(oo, Oc + ((size_t)i * Hq + h) * d, d * sizeof(double));
      } else {
        for (int c = 0; c < d; ++c) oo[c] = 0.0;
      }
      oracle_state_stream(qr + ((size_t)i * Hq + h) * d, kk, vv, keep, n, d,
                          scale, Bc, &mm, &ll, oo);
      for (int c = 0; c < d; ++c) oo[c] /= ll;
      lse[(size_t)i * Hq + h] = mm + log(ll);
      free(kk);
      free(vv);
      free(keep);
    }
  }
  free(pos);
  free(qr);
  free(kr);
}

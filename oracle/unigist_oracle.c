/*
 * UniGist attention oracle -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, fp64 CPU statement of what the gist-masked attention path
 * computes.  It is used by the tests, by the smoke check and by the CPU
 * baseline leg of the benchmark; the product library never links, loads or
 * calls anything in this directory, and this file shares no code, header,
 * table or constant with the CUDA path.
 *
 * Everything here works in the INTERLEAVED ("original") token order of the
 * paper's Eq. 2,
 *     Z = [sink_0..sink_{s-1}, x_0..x_{r-1}, g_0, x_r..x_{2r-1}, g_1, ...],
 * and evaluates the visibility rule of Eq. 3 token pair by token pair into an
 * explicit byte mask.  There is no tiling, no online softmax and no shifted
 * layout in here: softmax is "max, exp, sum, divide" over a whole row.
 *
 * All indices are 0-based.  s = sinks, T = raw tokens, r = compression ratio
 * (T % r == 0), n = T / r gists, N = s + T + n (Eq. 2's T'), k = number of
 * previous gist units in the local window (Section 4.1, text after Eq. 3).
 *
 * Parity pins (tests/test_oracle_*.py): literal set construction of Eq. 3,
 * closed-form row counts, dense causal attention when k >= n, row sums,
 * constant-V and zero-Q special cases, key-shift invariance, central finite
 * differences for the backward pass, brute-force "visible to any future
 * token" for compaction, decode == row of the full forward.
 *
 * Two readings of the paper are encoded here that no pin can settle, because
 * the paper prints no worked example for them (parity unpinned against the
 * authors' own implementation; every function is pinned against the paper's
 * equations as listed above): a window given as W raw tokens means
 * k = ceil(W / r) previous gist units (rounded up when r does not divide W),
 * and sink tokens belong to no gist unit, attend causally among themselves and
 * are seen by every later token.
 *
 * Functions take one (batch, KV-head) slice at a time: G query heads share
 * one K/V head (grouped-query attention, q head h uses kv head h / G).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { UG_SINK = 0, UG_RAW = 1, UG_GIST = 2 };

/* Eq. 2: classify interleaved position t.  unit = gist-unit number (raw and
 * gist tokens), number = index among tokens of the same kind. */
void ug_oracle_token(int64_t t, int64_t s, int64_t r, int32_t *kind,
                     int64_t *unit, int64_t *number) {
  if (t < s) {
    *kind = UG_SINK;
    *unit = -1;
    *number = t;
    return;
  }
  int64_t q = t - s;
  int64_t u = q / (r + 1);
  int64_t p = q % (r + 1);
  *unit = u;
  if (p == r) {
    *kind = UG_GIST;
    *number = u;
  } else {
    *kind = UG_RAW;
    *number = u * r + p;
  }
}

/* Eq. 3: A(z_t) = (S u G u W_t) n {j <= t}.  W_t = the gist unit holding z_t
 * plus the k units before it.  Sinks lie in no unit, so a sink query has an
 * empty W_t and sees earlier sinks only. */
int32_t ug_oracle_visible(int64_t t, int64_t j, int64_t s, int64_t r,
                          int64_t k) {
  if (j > t) return 0; /* autoregressive constraint */
  int32_t kt, kj;
  int64_t ut, uj, nt, nj;
  ug_oracle_token(t, s, r, &kt, &ut, &nt);
  ug_oracle_token(j, s, r, &kj, &uj, &nj);
  if (kj == UG_SINK) return 1; /* S */
  if (kj == UG_GIST) return 1; /* G */
  /* raw key: only through the local window W_t */
  if (kt == UG_SINK) return 0;
  return (uj >= ut - k) ? 1 : 0;
}

/* Rows [row_begin, row_end) of the N x N mask, one byte per pair. */
int32_t ug_oracle_mask(int64_t s, int64_t T, int64_t r, int64_t k,
                       int64_t row_begin, int64_t row_end, uint8_t *mask) {
  if (r <= 0 || T % r != 0 || s < 0 || k < 0) return 1;
  int64_t N = s + T + T / r;
  for (int64_t t = row_begin; t < row_end; ++t)
    for (int64_t j = 0; j < N; ++j)
      mask[(t - row_begin) * N + j] = (uint8_t)ug_oracle_visible(t, j, s, r, k);
  return 0;
}

/* Number of visible pairs in the whole mask (what "unmasked FLOPs" counts). */
int64_t ug_oracle_count_pairs(int64_t s, int64_t T, int64_t r, int64_t k) {
  int64_t N = s + T + T / r, c = 0;
  for (int64_t t = 0; t < N; ++t)
    for (int64_t j = 0; j <= t; ++j) c += ug_oracle_visible(t, j, s, r, k);
  return c;
}

/* Gist shift (Section 4.2): walk Z of Eq. 2, then move every gist to the
 * right end keeping the order inside each kind (a stable partition:
 * sinks, raw, gists).  shift_perm[sigma] = interleaved index of the token
 * that sits at shifted position sigma; unshift_perm is its inverse.
 * pos_ids (may be NULL) follows "position encoding alignment": a gist takes
 * the position id of the raw token right after it; ids count sinks and raw
 * tokens only. */
int32_t ug_oracle_layout(int64_t s, int64_t T, int64_t r, int32_t *shift_perm,
                         int32_t *unshift_perm, int32_t *pos_ids) {
  if (r <= 0 || T % r != 0 || s < 0) return 1;
  int64_t n = T / r, N = s + T + n;
  int8_t *kind = (int8_t *)malloc((size_t)N);
  int32_t *pos = (int32_t *)malloc((size_t)N * sizeof(int32_t));
  if (!kind || !pos) return 2;
  /* build Z literally */
  int64_t t = 0, next_pos = 0;
  for (int64_t i = 0; i < s; ++i) {
    kind[t] = UG_SINK;
    pos[t++] = (int32_t)next_pos++;
  }
  for (int64_t u = 0; u < n; ++u) {
    for (int64_t p = 0; p < r; ++p) {
      kind[t] = UG_RAW;
      pos[t++] = (int32_t)next_pos++;
    }
    kind[t] = UG_GIST;
    pos[t++] = (int32_t)next_pos; /* id of the raw token that follows */
  }
  int64_t sigma = 0;
  for (int pass = UG_SINK; pass <= UG_GIST; ++pass)
    for (int64_t i = 0; i < N; ++i)
      if (kind[i] == pass) shift_perm[sigma++] = (int32_t)i;
  for (int64_t i = 0; i < N; ++i) unshift_perm[shift_perm[i]] = (int32_t)i;
  if (pos_ids)
    for (int64_t i = 0; i < N; ++i) pos_ids[i] = pos[i];
  free(kind);
  free(pos);
  return 0;
}

static double dot(const double *a, const double *b, int D) {
  double acc = 0.0;
  for (int d = 0; d < D; ++d) acc += a[d] * b[d];
  return acc;
}

/*
 * Forward for one (batch, KV head) slice, rows [row_begin, row_end).
 *   q  [N][G][D], kk [N][D], v [N][D]   (interleaved order, fp64)
 *   o  [rows][G][D], lse [rows][G]
 * S_tj = scale * q_t . k_j on visible pairs, -inf elsewhere;
 * LSE_t = log sum_j exp(S_tj) (natural log); P = exp(S - LSE); O = P V.
 */
int32_t ug_oracle_attn_fwd(int64_t s, int64_t T, int64_t r, int64_t k,
                           int32_t G, int32_t D, double scale, const double *q,
                           const double *kk, const double *v,
                           int64_t row_begin, int64_t row_end, double *o,
                           double *lse) {
  if (r <= 0 || T % r != 0 || s < 0 || k < 0) return 1;
  const int64_t N = s + T + T / r;
  if (row_begin < 0 || row_end > N || row_begin > row_end) return 1;
  int32_t err = 0;
#pragma omp parallel
  {
    uint8_t *mrow = (uint8_t *)malloc((size_t)N);
    double *sc = (double *)malloc((size_t)N * sizeof(double));
    if (!mrow || !sc) {
#pragma omp atomic write
      err = 2;
    } else {
#pragma omp for schedule(dynamic, 4)
      for (int64_t t = row_begin; t < row_end; ++t) {
        for (int64_t j = 0; j < N; ++j)
          mrow[j] = (uint8_t)ug_oracle_visible(t, j, s, r, k);
        for (int32_t g = 0; g < G; ++g) {
          const double *qt = q + ((size_t)t * G + g) * D;
          double m = -INFINITY;
          for (int64_t j = 0; j < N; ++j) {
            if (!mrow[j]) continue;
            sc[j] = scale * dot(qt, kk + (size_t)j * D, D);
            if (sc[j] > m) m = sc[j];
          }
          double l = 0.0;
          for (int64_t j = 0; j < N; ++j)
            if (mrow[j]) l += exp(sc[j] - m);
          const double L = m + log(l);
          double *ot = o + ((size_t)(t - row_begin) * G + g) * D;
          for (int d = 0; d < D; ++d) ot[d] = 0.0;
          for (int64_t j = 0; j < N; ++j) {
            if (!mrow[j]) continue;
            const double p = exp(sc[j] - L);
            const double *vj = v + (size_t)j * D;
            for (int d = 0; d < D; ++d) ot[d] += p * vj[d];
          }
          lse[(size_t)(t - row_begin) * G + g] = L;
        }
      }
    }
    free(mrow);
    free(sc);
  }
  return err;
}

/*
 * Backward for one (batch, KV head) slice, restricted to a sample of outputs.
 *   q, dout [N][G][D]; kk, v [N][D].
 *   dq_out [n_rows][G][D] = dQ of the listed query rows,
 *   dk_out, dv_out [n_keys][D] = dK, dV of the listed key positions.
 * With P as in the forward:
 *   dV = P^T dO,  dP = dO V^T,  Delta_t = sum_j P_tj dP_tj,
 *   dS = P o (dP - Delta),  dQ = scale dS K,  dK = scale dS^T Q,
 * dK and dV summed over the G query heads of the slice.
 * Pass 1 walks the query rows that are listed or that see a listed key (LSE, Delta, dQ);
 * pass 2 walks the listed key columns and evaluates the column sums
 * dV_j = sum_t P_tj dO_t and dK_j = scale sum_t dS_tj q_t.
 */
int32_t ug_oracle_attn_bwd_sample(int64_t s, int64_t T, int64_t r, int64_t k,
                                  int32_t G, int32_t D, double scale,
                                  const double *q, const double *kk,
                                  const double *v, const double *dout,
                                  int64_t n_rows, const int64_t *rows,
                                  int64_t n_keys, const int64_t *keys,
                                  double *dq_out, double *dk_out,
                                  double *dv_out) {
  if (r <= 0 || T % r != 0 || s < 0 || k < 0) return 1;
  const int64_t N = s + T + T / r;
  double *lse = (double *)malloc((size_t)N * G * sizeof(double));
  double *delta = (double *)malloc((size_t)N * G * sizeof(double));
  int64_t *slot = (int64_t *)malloc((size_t)N * sizeof(int64_t)); /* -1, -2 or dq slot */
  if (!lse || !delta || !slot) return 2;
  for (int64_t t = 0; t < N; ++t) slot[t] = -1; /* not needed */
  for (int64_t a = 0; a < n_keys; ++a) {
    if (keys[a] < 0 || keys[a] >= N) return 1;
    for (int64_t t = keys[a]; t < N; ++t)
      if (ug_oracle_visible(t, keys[a], s, r, k)) slot[t] = -2; /* needed, no dq */
  }
  for (int64_t a = 0; a < n_rows; ++a) {
    if (rows[a] < 0 || rows[a] >= N) return 1;
    slot[rows[a]] = a;
  }
  int32_t err = 0;
#pragma omp parallel
  {
    uint8_t *mrow = (uint8_t *)malloc((size_t)N);
    double *sc = (double *)malloc((size_t)N * sizeof(double));
    double *dp = (double *)malloc((size_t)N * sizeof(double));
    if (!mrow || !sc || !dp) {
#pragma omp atomic write
      err = 2;
    } else {
#pragma omp for schedule(dynamic, 4)
      for (int64_t t = 0; t < N; ++t) {
        if (slot[t] == -1) continue;
        for (int64_t j = 0; j < N; ++j)
          mrow[j] = (uint8_t)ug_oracle_visible(t, j, s, r, k);
        for (int32_t g = 0; g < G; ++g) {
          const double *qt = q + ((size_t)t * G + g) * D;
          const double *dot_ = dout + ((size_t)t * G + g) * D;
          double m = -INFINITY;
          for (int64_t j = 0; j < N; ++j) {
            if (!mrow[j]) continue;
            sc[j] = scale * dot(qt, kk + (size_t)j * D, D);
            if (sc[j] > m) m = sc[j];
          }
          double l = 0.0;
          for (int64_t j = 0; j < N; ++j)
            if (mrow[j]) l += exp(sc[j] - m);
          const double L = m + log(l);
          double dl = 0.0;
          for (int64_t j = 0; j < N; ++j) {
            if (!mrow[j]) continue;
            sc[j] = exp(sc[j] - L); /* now P_tj */
            dp[j] = dot(dot_, v + (size_t)j * D, D);
            dl += sc[j] * dp[j];
          }
          lse[(size_t)t * G + g] = L;
          delta[(size_t)t * G + g] = dl;
          if (slot[t] < 0) continue;
          double *dqt = dq_out + ((size_t)slot[t] * G + g) * D;
          for (int d = 0; d < D; ++d) dqt[d] = 0.0;
          for (int64_t j = 0; j < N; ++j) {
            if (!mrow[j]) continue;
            const double ds = sc[j] * (dp[j] - dl);
            const double *kj = kk + (size_t)j * D;
            for (int d = 0; d < D; ++d) dqt[d] += scale * ds * kj[d];
          }
        }
      }
    }
    free(mrow);
    free(sc);
    free(dp);
  }
  if (!err) {
#pragma omp parallel for schedule(dynamic, 1)
    for (int64_t a = 0; a < n_keys; ++a) {
      const int64_t j = keys[a];
      double *dkj = dk_out + (size_t)a * D;
      double *dvj = dv_out + (size_t)a * D;
      const double *kj = kk + (size_t)j * D;
      const double *vj = v + (size_t)j * D;
      for (int d = 0; d < D; ++d) dkj[d] = dvj[d] = 0.0;
      for (int64_t t = j; t < N; ++t) {
        if (!ug_oracle_visible(t, j, s, r, k)) continue;
        for (int32_t g = 0; g < G; ++g) {
          const double *qt = q + ((size_t)t * G + g) * D;
          const double *dot_ = dout + ((size_t)t * G + g) * D;
          const double p =
              exp(scale * dot(qt, kj, D) - lse[(size_t)t * G + g]);
          const double ds =
              p * (dot(dot_, vj, D) - delta[(size_t)t * G + g]);
          for (int d = 0; d < D; ++d) {
            dvj[d] += p * dot_[d];
            dkj[d] += scale * ds * qt[d];
          }
        }
      }
    }
  }
  free(lse);
  free(delta);
  free(slot);
  return err;
}

/* The whole backward of one slice: every row and every key.
 *   dq [N][G][D]; dk, dv [N][D]. */
int32_t ug_oracle_attn_bwd(int64_t s, int64_t T, int64_t r, int64_t k,
                           int32_t G, int32_t D, double scale, const double *q,
                           const double *kk, const double *v,
                           const double *dout, double *dq, double *dk,
                           double *dv) {
  if (r <= 0 || T % r != 0 || s < 0 || k < 0) return 1;
  const int64_t N = s + T + T / r;
  int64_t *all = (int64_t *)malloc((size_t)N * sizeof(int64_t));
  if (!all) return 2;
  for (int64_t t = 0; t < N; ++t) all[t] = t;
  int32_t rc = ug_oracle_attn_bwd_sample(s, T, r, k, G, D, scale, q, kk, v, dout,
                                         N, all, N, all, dq, dk, dv);
  free(all);
  return rc;
}

/*
 * Compaction (Section 4.3, flexible inference): right after the last gist of
 * a T-token prefix has been inserted, a cached token may be dropped iff no
 * FUTURE token can ever see it.  Brute force: extend the sequence by k + 2
 * more gist units and keep j < N iff some t >= N has visible(t, j).
 * kept[] lists the survivors as interleaved indices in cache order: sinks,
 * then gists ascending, then raw ascending.  Returns the count (<0 on error).
 */
int64_t ug_oracle_kept_set(int64_t s, int64_t T, int64_t r, int64_t k,
                           int32_t *kept) {
  if (r <= 0 || T % r != 0 || s < 0 || k < 0) return -1;
  const int64_t N = s + T + T / r;
  const int64_t N_ext = N + (k + 2) * (r + 1);
  uint8_t *keep = (uint8_t *)calloc((size_t)N, 1);
  if (!keep) return -2;
  for (int64_t j = 0; j < N; ++j)
    for (int64_t t = N; t < N_ext && !keep[j]; ++t)
      if (ug_oracle_visible(t, j, s, r, k)) keep[j] = 1;
  int64_t c = 0;
  for (int pass = UG_SINK; pass <= UG_GIST; ++pass) {
    /* cache order: sinks, gists, raw */
    const int want = (pass == 0) ? UG_SINK : (pass == 1 ? UG_GIST : UG_RAW);
    for (int64_t j = 0; j < N; ++j) {
      int32_t kd;
      int64_t u, nn;
      ug_oracle_token(j, s, r, &kd, &u, &nn);
      if (kd == want && keep[j]) kept[c++] = (int32_t)j;
    }
  }
  free(keep);
  return c;
}

/*
 * Decode: G query heads of one KV head attend to ALL L cache entries
 * (whatever is still in a compacted cache is visible by construction).
 *   qd [G][D], kc [L][D], vc [L][D] -> o [G][D], lse [G].
 */
int32_t ug_oracle_decode(int64_t L, int32_t G, int32_t D, double scale,
                         const double *qd, const double *kc, const double *vc,
                         double *o, double *lse) {
  if (L <= 0) return 1;
  double *sc = (double *)malloc((size_t)L * sizeof(double));
  if (!sc) return 2;
  for (int32_t g = 0; g < G; ++g) {
    double m = -INFINITY;
    for (int64_t j = 0; j < L; ++j) {
      sc[j] = scale * dot(qd + (size_t)g * D, kc + (size_t)j * D, D);
      if (sc[j] > m) m = sc[j];
    }
    double l = 0.0;
    for (int64_t j = 0; j < L; ++j) l += exp(sc[j] - m);
    const double Lg = m + log(l);
    for (int d = 0; d < D; ++d) o[(size_t)g * D + d] = 0.0;
    for (int64_t j = 0; j < L; ++j) {
      const double p = exp(sc[j] - Lg);
      for (int d = 0; d < D; ++d) o[(size_t)g * D + d] += p * vc[(size_t)j * D + d];
    }
    lse[g] = Lg;
  }
  free(sc);
  return 0;
}

int32_t ug_oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/*
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * Plain fp64 CPU oracle for the fused-attention forward pass. Only the test
 * suite, the smoke check and the benchmark's cpu_baseline / reference arm may
 * call it. It shares no code, header, table or helper with the CUDA path.
 *
 * What it computes is the definition itself (the paper's attention equation,
 * Section "Fused Attention":  R = softmax(Q K^T / sqrt(d)) V ), written out
 * row by row, because the fused method reaches exactly that result up to
 * rounding order.  For every (batch, head) and every requested row i:
 *
 *     s_j   = (sum_c q_ic * k_jc) * (1/sqrt(d))          j = 0..L-1
 *     M     = max_j s_j
 *     p_j   = exp(s_j - M)            (the max shift is value-neutral,
 *                                      Section "Online Softmax")
 *     delta = sum_j p_j
 *     o_c   = (sum_j p_j * v_jc) / delta
 *
 * Inputs are bf16 bit patterns (uint16), widened exactly to fp64; every
 * operation is fp64; the result is returned in fp64.  There is no blocking,
 * no fusion and no streaming: one row at a time, one pass per formula line.
 *
 * Pins (tests, CPU only): identical-V rows, Q = 0 column mean, softmax rows
 * summing to one, no-max-shift brute force on tiny L, L = 1 and L = 2 closed
 * forms, permutation / key-shift / linearity invariants, structured
 * identity-matrix cases, and agreement with scipy's softmax + numpy matmul.
 * The paper prints no numeric attention outputs, so parity with the paper's
 * own outputs is unpinned.
 *
 * Causal variant (attn_oracle_rows_causal): the same definition with the scores of
 * keys after the query's own position set to -inf before the softmax (the
 * paper's boundary rule -- masked elements are -inf, never zero -- applied to a
 * triangular mask), i.e. row i attends to keys 0..i only.  Pinned by: row i
 * equals the non-causal result over the first i+1 keys; row 0 equals V[0];
 * changing K/V rows after position i leaves row i unchanged.
 *
 * Layout: q, k, v are contiguous [B][H][L][d], d fastest.
 * rows[]: n_rows row indices in [0, L), the same list for every head.
 * out:    [B*H][n_rows][d] fp64.
 * psum:   optional [B*H][n_rows] fp64, receives sum_j p_j / delta (== 1).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

static double bf16_to_f64(uint16_t h) {
  uint32_t bits = ((uint32_t)h) << 16; /* bf16 is the top half of an fp32 */
  float f;
  memcpy(&f, &bits, sizeof f);
  return (double)f;
}

int attn_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

static int oracle_rows_impl(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                            int B, int H, int L, int d, const int32_t *rows,
                            int n_rows, double *out, double *psum, int causal) {
  if (!q || !k || !v || !rows || !out) return -1;
  if (B <= 0 || H <= 0 || L <= 0 || d <= 0 || n_rows < 0) return -1;
  for (int r = 0; r < n_rows; ++r)
    if (rows[r] < 0 || rows[r] >= L) return -2;

  const double inv_sqrt_d = 1.0 / sqrt((double)d);
  const size_t head_elems = (size_t)L * (size_t)d;
  int status = 0;

  for (int bh = 0; bh < B * H; ++bh) {
    /* widen this head's K and V once (exact) */
    double *Kd = (double *)malloc(head_elems * sizeof(double));
    double *Vd = (double *)malloc(head_elems * sizeof(double));
    if (!Kd || !Vd) {
      free(Kd);
      free(Vd);
      return -3;
    }
    const uint16_t *kh = k + (size_t)bh * head_elems;
    const uint16_t *vh = v + (size_t)bh * head_elems;
    const uint16_t *qh = q + (size_t)bh * head_elems;
    for (size_t e = 0; e < head_elems; ++e) {
      Kd[e] = bf16_to_f64(kh[e]);
      Vd[e] = bf16_to_f64(vh[e]);
    }

#pragma omp parallel
    {
      double *s = (double *)malloc((size_t)L * sizeof(double));
      double *qi = (double *)malloc((size_t)d * sizeof(double));
      double *acc = (double *)malloc((size_t)d * sizeof(double));
      if (!s || !qi || !acc) {
#pragma omp atomic write
        status = -3;
      } else {
#pragma omp for schedule(dynamic, 1)
        for (int r = 0; r < n_rows; ++r) {
          const int i = rows[r];
          for (int c = 0; c < d; ++c) qi[c] = bf16_to_f64(qh[(size_t)i * d + c]);

          /* keys this row may attend to: all of them, or 0..i when causal */
          const int Lk = causal ? i + 1 : L;
          /* scores and their maximum */
          double M = -INFINITY;
          for (int j = 0; j < Lk; ++j) {
            const double *kj = Kd + (size_t)j * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += qi[c] * kj[c];
            s[j] = dot * inv_sqrt_d;
            if (s[j] > M) M = s[j];
          }
          /* weights and normaliser */
          double delta = 0.0;
          for (int j = 0; j < Lk; ++j) {
            s[j] = exp(s[j] - M);
            delta += s[j];
          }
          /* weighted sum of value rows */
          for (int c = 0; c < d; ++c) acc[c] = 0.0;
          for (int j = 0; j < Lk; ++j) {
            const double pj = s[j];
            const double *vj = Vd + (size_t)j * d;
            for (int c = 0; c < d; ++c) acc[c] += pj * vj[c];
          }
          double *o = out + ((size_t)bh * n_rows + r) * d;
          for (int c = 0; c < d; ++c) o[c] = acc[c] / delta;
          if (psum) {
            double t = 0.0;
            for (int j = 0; j < Lk; ++j) t += s[j] / delta;
            psum[(size_t)bh * n_rows + r] = t;
          }
        }
      }
      free(s);
      free(qi);
      free(acc);
    }
    free(Kd);
    free(Vd);
    if (status) return status;
  }
  return 0;
}

int attn_oracle_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                     int B, int H, int L, int d, const int32_t *rows,
                     int n_rows, double *out, double *psum) {
  return oracle_rows_impl(q, k, v, B, H, L, d, rows, n_rows, out, psum, 0);
}

int attn_oracle_rows_causal(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                            int B, int H, int L, int d, const int32_t *rows,
                            int n_rows, double *out, double *psum) {
  return oracle_rows_impl(q, k, v, B, H, L, d, rows, n_rows, out, psum, 1);
}

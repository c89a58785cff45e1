/*
 * CPU ORACLE -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision restatement of what one suffix-pruned
 * block-diffusion denoising step computes.  Only tests, the smoke check and the
 * benchmark's CPU-baseline leg may call it; the CUDA library shares no code
 * with it.  Nothing here is blocked, fused or reordered beyond the paper's
 * definitions, so every function can be checked against the cited passage by
 * eye.  OpenMP is used only over independent (batch, head) pairs, logit rows
 * and sequences.
 *
 *   oracle_attn        Method, "Attenuation Guided Suffix Modeling" (Eq. 7, 8)
 *                      and the query/key construction of "Dynamic Confidence
 *                      Aware Parallel Decoding": softmax attention of the
 *                      retained rows over [cached prefix ; retained rows].
 *   oracle_confidence  Preliminary, Eq. 4: c = max softmax(z), x^ = argmax.
 *   oracle_select      Eq. 9 (selection rule), Eq. 10 (adaptive threshold),
 *                      Eq. 5 (state update), block termination test and the
 *                      "Early Exit For Block Diffusion" paragraph.
 *
 * All arrays are dense, row-major, contiguous.  Inputs are float32 (bf16
 * values are widened exactly by the caller); attention and confidence
 * accumulate in double.  The selection rule is evaluated in float32, one
 * rounding per operation (compile with -ffp-contract=off), because its
 * threshold decides integers.
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

/*
 * Pruned bidirectional attention (Eq. 8 input x~ = prefix U current U pruned
 * suffix; queries = current U pruned suffix; keys/values = all of x~, the
 * prefix part read from the cache).
 *
 *   q_tail           [B][Hq ][T][D]   queries of the whole tail (block + suffix)
 *   k_tail, v_tail   [B][Hkv][T][D]
 *   k_pre,  v_pre    [B][Hkv][P][D]   cached prefix keys / values
 *   idx              [Lq] when idx_bstride == 0, else [B][Lq] with that stride;
 *                    retained tail rows (Eq. 7), values in [0, T)
 *   out              [B][Hq][Lq][D]   double
 *   lse              [B][Hq][Lq]      natural-log sum-exp of the scaled scores,
 *                                     may be NULL
 *
 * Query head hq reads KV head hq / (Hq / Hkv).  No mask of any kind: the
 * model is bidirectional.  Returns 0, or -1 on a bad argument.
 */
int oracle_attn(const float *q_tail, const float *k_tail, const float *v_tail,
                const float *k_pre, const float *v_pre, int B, int Hq, int Hkv,
                int D, int P, int T, int Lq, const int32_t *idx,
                long idx_bstride, double scale, double *out, double *lse) {
  if (B < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv != 0 || D <= 0 || P < 0 ||
      T < 0 || Lq < 0 || Lq > T)
    return -1;
  const int G = Hq / Hkv;
  const int Lkv = P + Lq;
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < Lq; ++i) {
      int r = idx[(long)b * idx_bstride + i];
      if (r < 0 || r >= T) return -1;
    }
  int bad = 0;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b)
    for (int hq = 0; hq < Hq; ++hq) {
      const int hk = hq / G;
      const int32_t *ix = idx + (long)b * idx_bstride;
      const float *Qt = q_tail + ((long)b * Hq + hq) * T * D;
      const float *Kt = k_tail + ((long)b * Hkv + hk) * T * D;
      const float *Vt = v_tail + ((long)b * Hkv + hk) * T * D;
      const float *Kp = k_pre + ((long)b * Hkv + hk) * P * D;
      const float *Vp = v_pre + ((long)b * Hkv + hk) * P * D;
      double *s = (double *)malloc(sizeof(double) * (Lkv > 0 ? Lkv : 1));
      if (!s) {
        bad = 1;
        continue;
      }
      for (int i = 0; i < Lq; ++i) {
        const float *q = Qt + (long)ix[i] * D;
        double m = -INFINITY;
        for (int j = 0; j < Lkv; ++j) {
          const float *k = (j < P) ? Kp + (long)j * D : Kt + (long)ix[j - P] * D;
          double acc = 0.0;
          for (int d = 0; d < D; ++d) acc += (double)q[d] * (double)k[d];
          s[j] = scale * acc;
          if (s[j] > m) m = s[j];
        }
        double l = 0.0;
        for (int j = 0; j < Lkv; ++j) {
          s[j] = exp(s[j] - m);
          l += s[j];
        }
        double *o = out + (((long)b * Hq + hq) * Lq + i) * D;
        for (int d = 0; d < D; ++d) o[d] = 0.0;
        for (int j = 0; j < Lkv; ++j) {
          const float *v = (j < P) ? Vp + (long)j * D : Vt + (long)ix[j - P] * D;
          const double p = s[j] / l;
          for (int d = 0; d < D; ++d) o[d] += p * (double)v[d];
        }
        if (lse) lse[((long)b * Hq + hq) * Lq + i] = m + log(l);
      }
      free(s);
    }
  return bad ? -2 : 0;
}

/*
 * Eq. 4: for every row of logits z, c = max_j softmax(z)_j = 1 / sum_j
 * exp(z_j - max z), and x^ = argmax_j z_j.  Equal maxima resolve to the
 * lowest index.  logits [rows][V] float32 with row stride ld >= V.
 */
int oracle_confidence(const float *logits, long rows, long V, long ld,
                      double *conf, int32_t *tok) {
  if (rows < 0 || V <= 0 || ld < V) return -1;
#pragma omp parallel for schedule(static)
  for (long r = 0; r < rows; ++r) {
    const float *z = logits + r * ld;
    double m = (double)z[0];
    long arg = 0;
    for (long j = 1; j < V; ++j)
      if ((double)z[j] > m) {
        m = (double)z[j];
        arg = j;
      }
    double sum = 0.0;
    for (long j = 0; j < V; ++j) sum += exp((double)z[j] - m);
    conf[r] = 1.0 / sum;
    tok[r] = (int32_t)arg;
  }
  return 0;
}

/*
 * Eq. 10 in float32, one rounding per operation:
 *   r_mask = (n_masked + extra) / (K + extra)
 *   tau    = tau0 * (1 - alpha * (1 - r_mask))
 * extra = 0 counts the block only; extra = R counts the (all still masked)
 * retained suffix rows of the query as well.
 */
float oracle_threshold(int n_masked, int K, int extra, float tau0, float alpha) {
  volatile float r = (float)(n_masked + extra) / (float)(K + extra);
  volatile float t1 = 1.0f - r;
  volatile float t2 = alpha * t1;
  volatile float t3 = 1.0f - t2;
  volatile float tau = tau0 * t3;
  return tau;
}

/*
 * One selection step for every listed sequence (Eq. 9, 10, 5).
 *
 *   conf, tok        [B][K]   from Eq. 4
 *   masked           [B][K]   in/out, 1 = position still holds MASK
 *   x_block          [B][K]   in/out token ids of the current block
 *   seq_list         n_seq sequence numbers to process, or NULL = all B
 *   sel_idx          [B][K]   accepted positions, ascending; the rest -1
 *   sel_cnt          [B]
 *   block_done       [B]      1 when no MASK is left in the block
 *   eos_exit         [B]      in/out, OR-ed: an accepted token equals eos_id
 *                             with confidence >= eos_tau (eos_id < 0: never)
 *   active_seq       [B]      processed sequences whose block still has
 *                             masks, ascending; *active_cnt their number
 *
 * Rule: with n masked positions (counted before the update), tau from Eq. 10;
 * accept every masked position with conf >= tau; when none qualifies accept
 * the single masked position of highest confidence (lowest index among equal
 * ones); n == 0 accepts nothing.  Unlisted sequences are left untouched.
 */
int oracle_select(int B, int K, const float *conf, const int32_t *tok,
                  uint8_t *masked, int32_t *x_block, float tau0, float alpha,
                  int ratio_extra, int eos_id, float eos_tau,
                  const int32_t *seq_list, int n_seq, int32_t *sel_idx,
                  int32_t *sel_cnt, uint8_t *block_done, uint8_t *eos_exit,
                  int32_t *active_seq, int32_t *active_cnt, float *tau_out) {
  if (B < 0 || K <= 0 || ratio_extra < 0) return -1;
  const int n = seq_list ? n_seq : B;
  if (n < 0 || n > B) return -1;
  int n_active = 0;
  for (int s = 0; s < n; ++s) {
    const int b = seq_list ? seq_list[s] : s;
    if (b < 0 || b >= B) return -1;
    if (s > 0 && seq_list && seq_list[s - 1] >= b) return -1; /* ascending */
    const float *c = conf + (long)b * K;
    const int32_t *t = tok + (long)b * K;
    uint8_t *mk = masked + (long)b * K;
    int32_t *x = x_block + (long)b * K;
    int32_t *si = sel_idx + (long)b * K;
    int nm = 0;
    for (int i = 0; i < K; ++i) nm += mk[i] ? 1 : 0;
    for (int i = 0; i < K; ++i) si[i] = -1;
    int cnt = 0;
    float tau = oracle_threshold(nm, K, ratio_extra, tau0, alpha);
    if (tau_out) tau_out[b] = tau;
    if (nm > 0) {
      for (int i = 0; i < K; ++i)
        if (mk[i] && c[i] >= tau) si[cnt++] = i;
      if (cnt == 0) {
        int best = -1;
        for (int i = 0; i < K; ++i)
          if (mk[i] && (best < 0 || c[i] > c[best])) best = i;
        si[cnt++] = best;
      }
    }
    int eos = 0;
    for (int k = 0; k < cnt; ++k) {
      const int i = si[k];
      x[i] = t[i];
      mk[i] = 0;
      if (eos_id >= 0 && t[i] == eos_id && c[i] >= eos_tau) eos = 1;
    }
    sel_cnt[b] = cnt;
    const int done = (nm - cnt) == 0;
    block_done[b] = (uint8_t)done;
    if (eos) eos_exit[b] = 1;
    if (!done) active_seq[n_active++] = b;
  }
  *active_cnt = n_active;
  return 0;
}

/*
 * Output projection followed by Eq. 4, without storing the logits.
 *
 * After the attention, the rest of the model turns the hidden states into the
 * prediction logits (Method, "Dynamic Confidence Aware Parallel Decoding");
 * the last of those components is the output projection z_r = W h_r.  Eq. 4 then reads c_r = max_j
 * softmax(z_r)_j and x^_r = argmax_j z_rj.  This function is that composition
 * written out: a plain matrix-vector product in double per row, then the same
 * max / lowest-index argmax / sum of exponentials as oracle_confidence.
 *
 *   hidden  [rows][hid]  float32 (bf16 values widened exactly by the caller)
 *   weight  [V][hid]     float32, row j is the output embedding of token j
 *   conf    [rows]       double
 *   tok     [rows]
 *   logits  [rows][V]    double, may be NULL
 */
int oracle_lmhead_confidence(const float *hidden, const float *weight, long rows,
                             long hid, long V, double *conf, int32_t *tok,
                             double *logits) {
  if (rows < 0 || hid <= 0 || V <= 0) return -1;
  int bad = 0;
#pragma omp parallel for schedule(dynamic, 1)
  for (long r = 0; r < rows; ++r) {
    const float *h = hidden + r * hid;
    double *z = logits ? logits + r * V : (double *)malloc(sizeof(double) * V);
    if (!z) {
      bad = 1;
      continue;
    }
    for (long j = 0; j < V; ++j) {
      const float *w = weight + j * hid;
      double acc = 0.0;
      for (long k = 0; k < hid; ++k) acc += (double)h[k] * (double)w[k];
      z[j] = acc;
    }
    double m = z[0];
    long arg = 0;
    for (long j = 1; j < V; ++j)
      if (z[j] > m) {
        m = z[j];
        arg = j;
      }
    double sum = 0.0;
    for (long j = 0; j < V; ++j) sum += exp(z[j] - m);
    conf[r] = 1.0 / sum;
    tok[r] = (int32_t)arg;
    if (!logits) free(z);
  }
  return bad ? -2 : 0;
}

/*
 * Rotary position encoding of the retained rows with their ORIGINAL position
 * ids, and their gather into compact buffers (Method, "Attenuation Guided
 * Suffix Modeling": pruned tokens keep their place in the sequence through
 * their rotary position ids; Eq. 7 names the retained set, Eq. 8 the pruned
 * input).
 *
 * For every batch b, head h and retained row i (tail row r = idx[i], absolute
 * position p = pos_offset + r), with half = D / 2 and, for d < half,
 * angle = p * theta^(-2 d / D):
 *     out[d]        = x[d] cos(angle) - x[d + half] sin(angle)
 *     out[d + half] = x[d + half] cos(angle) + x[d] sin(angle)
 * (the "rotate half" pairing of dimension d with d + D/2).  Q and K are
 * rotated, V is only gathered.
 *
 *   q_raw           [B][Hq ][T][D]   float32 (bf16 widened exactly)
 *   k_raw, v_raw    [B][Hkv][T][D]
 *   idx             [Lq] (idx_bstride 0) or [B][Lq]
 *   q_out           [B][Hq ][Lq][D]  double
 *   k_out, v_out    [B][Hkv][Lq][D]  double
 */
int oracle_rope_gather(const float *q_raw, const float *k_raw, const float *v_raw,
                       int B, int Hq, int Hkv, int D, int T, int Lq,
                       const int32_t *idx, long idx_bstride, long pos_offset,
                       double theta, double *q_out, double *k_out, double *v_out) {
  if (B < 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || (D & 1) || T < 0 || Lq < 0 || theta <= 0.0) return -1;
  const int half = D / 2;
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < Lq; ++i) {
      const int r = idx[(long)b * idx_bstride + i];
      if (r < 0 || r >= T) return -1;
    }
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < Lq; ++i) {
      const int r = idx[(long)b * idx_bstride + i];
      const double p = (double)(pos_offset + r);
      for (int which = 0; which < 2; ++which) {       /* 0: queries, 1: keys */
        const int H = which ? Hkv : Hq;
        const float *src = which ? k_raw : q_raw;
        double *dst = which ? k_out : q_out;
        for (int h = 0; h < H; ++h) {
          const float *x = src + (((long)b * H + h) * T + r) * D;
          double *o = dst + (((long)b * H + h) * Lq + i) * D;
          for (int d = 0; d < half; ++d) {
            const double angle = p * pow(theta, -2.0 * (double)d / (double)D);
            const double c = cos(angle), s = sin(angle);
            o[d] = (double)x[d] * c - (double)x[d + half] * s;
            o[d + half] = (double)x[d + half] * c + (double)x[d] * s;
          }
        }
      }
      for (int h = 0; h < Hkv; ++h) {
        const float *x = v_raw + (((long)b * Hkv + h) * T + r) * D;
        double *o = v_out + (((long)b * Hkv + h) * Lq + i) * D;
        for (int d = 0; d < D; ++d) o[d] = (double)x[d];
      }
    }
  return 0;
}

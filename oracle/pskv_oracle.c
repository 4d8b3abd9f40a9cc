/*
 * fp64 CPU oracle for shared-prefix batched causal attention.
 *
 * TEST INFRASTRUCTURE ONLY.  Nothing on the product path may call, link or
 * import this file; it exists so that the CUDA kernels can be compared with
 * an independent, slow, obviously-correct program.  It shares no code with
 * the CUDA path.
 *
 * What it computes (paper Sec. 3, Eq. 2 with the cache of Eq. 3):
 *   every candidate b gets its OWN physical copy of the prefix keys/values
 *   (the "Repeat(K, V, times = N)" of Eq. 3, i.e. the standard-KV-cache
 *   formulation), the candidate's suffix keys/values are appended
 *   (Sec. 4.2: the prefix cache is concatenated with the suffix-side K/V
 *   of the current layer), and ordinary causal scaled-dot-product attention
 *   (Eq. 2) is run for the S suffix-side query rows: row i sees the P
 *   prefix keys and suffix keys 0..i.
 *
 *   Grouped-query attention (Appendix E: several query heads share one KV
 *   head): query head h reads KV head g = h / (Hq / Hkv).
 *
 * Layouts (dense, row-major, last index fastest), all fp64:
 *   q, out, dout, dq     [B][Hq][S][d]
 *   prefix_k, prefix_v   [Hkv][P][d]
 *   suffix_k, suffix_v   [B][Hkv][S][d]      (also dk_suffix, dv_suffix)
 *   lse                  [B][Hq][S]          natural log of sum_j exp(s_j)
 *
 * Parity pins (tests/test_oracle_pins.py): full-sequence no-cache attention
 * through a library routine, closed forms (zero queries, constant values,
 * key shift, the P=1,S=1 logistic form), prefix/suffix split invariance,
 * candidate permutation, GQA-vs-repeated-MHA, the log-sum-exp merge
 * identity, and central finite differences for the backward pass.
 */
#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

int pskv_oracle_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* K_full[b,g] = prefix_k[g] (+) suffix_k[b,g]  -- the per-candidate physical
 * duplicate of Eq. 3, followed by the concatenation of Sec. 4.2. */
static void build_full_kv(const double *prefix, const double *suffix, double *full,
                          int b, int g, int Hkv, int S, int P, int d)
{
    memcpy(full, prefix + (size_t)g * P * d, sizeof(double) * (size_t)P * d);
    memcpy(full + (size_t)P * d, suffix + ((size_t)b * Hkv + g) * S * d,
           sizeof(double) * (size_t)S * d);
}

/* Eq. 2 for one query row against its n_vis visible keys.
 * s[j] = scale * <q, K[j]>, returns lse = m + ln sum exp(s - m) and leaves
 * the normalised probabilities in p[0..n_vis). */
static double softmax_row(const double *qrow, const double *K, int n_vis, int d,
                          double scale, double *p)
{
    double m = -INFINITY;
    for (int j = 0; j < n_vis; ++j) {
        double acc = 0.0;
        for (int c = 0; c < d; ++c) acc += qrow[c] * K[(size_t)j * d + c];
        p[j] = scale * acc;
        if (p[j] > m) m = p[j];
    }
    double l = 0.0;
    for (int j = 0; j < n_vis; ++j) {
        p[j] = exp(p[j] - m);
        l += p[j];
    }
    for (int j = 0; j < n_vis; ++j) p[j] /= l;
    return m + log(l);
}

int pskv_oracle_attn_fwd(const double *q, const double *prefix_k, const double *prefix_v,
                         const double *suffix_k, const double *suffix_v, double scale,
                         double *out, double *lse,
                         int B, int Hq, int Hkv, int S, int P, int d)
{
    if (B < 1 || Hq < 1 || Hkv < 1 || S < 1 || P < 0 || d < 1 || Hq % Hkv != 0) return 1;
    const int n_rep = Hq / Hkv;
    const int T = P + S;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        if (!Kf || !Vf || !p) {
            failed = 1;
        } else {
            for (int g = 0; g < Hkv; ++g) {
                build_full_kv(prefix_k, suffix_k, Kf, b, g, Hkv, S, P, d);
                build_full_kv(prefix_v, suffix_v, Vf, b, g, Hkv, S, P, d);
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < S; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * S + i;
                        const int n_vis = P + i + 1;
                        lse[row] = softmax_row(q + row * d, Kf, n_vis, d, scale, p);
                        double *o = out + row * d;
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
    }
    return failed ? 2 : 0;
}

/*
 * Closed-form backward of L = sum(out * dout) (no autodiff).  From the
 * softmax Jacobian d o / d s_j = p_j (v_j - o):
 *   D    = <dout_row, out_row>
 *   dp_j = <dout_row, V[j]>
 *   ds_j = p_j (dp_j - D)
 *   dq_row        = scale * sum_j ds_j K[j]
 *   dK[j]        += scale * ds_j q_row          (kept only for suffix keys j >= P)
 *   dV[j]        += p_j dout_row                (kept only for suffix keys j >= P)
 * Suffix-key gradients are summed over the query rows that see the key and
 * over the Hq/Hkv query heads that share the KV head.  The prefix cache is
 * computed once and frozen (Sec. 4.2: only gradients with respect to the
 * suffix side are needed), so contributions to prefix keys are discarded.
 * The forward quantities (p, out) are recomputed here in fp64.
 */
static int attn_bwd_impl(const double *dout, const double *dlse, const double *q,
                         const double *prefix_k, const double *prefix_v,
                         const double *suffix_k, const double *suffix_v, double scale,
                         double *dq, double *dk_suffix, double *dv_suffix,
                         int B, int Hq, int Hkv, int S, int P, int d)
{
    if (B < 1 || Hq < 1 || Hkv < 1 || S < 1 || P < 0 || d < 1 || Hq % Hkv != 0) return 1;
    const int n_rep = Hq / Hkv;
    const int T = P + S;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        if (!Kf || !Vf || !p || !o) {
            failed = 1;
        } else {
            for (int g = 0; g < Hkv; ++g) {
                build_full_kv(prefix_k, suffix_k, Kf, b, g, Hkv, S, P, d);
                build_full_kv(prefix_v, suffix_v, Vf, b, g, Hkv, S, P, d);
                double *dKs = dk_suffix + ((size_t)b * Hkv + g) * S * d;
                double *dVs = dv_suffix + ((size_t)b * Hkv + g) * S * d;
                for (size_t e = 0; e < (size_t)S * d; ++e) { dKs[e] = 0.0; dVs[e] = 0.0; }
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < S; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * S + i;
                        const int n_vis = P + i + 1;
                        const double *qr = q + row * d;
                        const double *go = dout + row * d;
                        softmax_row(qr, Kf, n_vis, d, scale, p);
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                        double D = 0.0;
                        for (int c = 0; c < d; ++c) D += go[c] * o[c];
                        const double gl = dlse ? dlse[row] : 0.0;  /* d lse / d s_j = p_j */
                        double *dqr = dq + row * d;
                        for (int c = 0; c < d; ++c) dqr[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j) {
                            double dp = 0.0;
                            for (int c = 0; c < d; ++c) dp += go[c] * Vf[(size_t)j * d + c];
                            const double ds = p[j] * (dp - D + gl);
                            for (int c = 0; c < d; ++c) dqr[c] += scale * ds * Kf[(size_t)j * d + c];
                            if (j >= P) {
                                const int t = j - P;
                                for (int c = 0; c < d; ++c) {
                                    dKs[(size_t)t * d + c] += scale * ds * qr[c];
                                    dVs[(size_t)t * d + c] += p[j] * go[c];
                                }
                            }
                        }
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
        free(o);
    }
    return failed ? 2 : 0;
}

int pskv_oracle_attn_bwd(const double *dout, const double *q,
                         const double *prefix_k, const double *prefix_v,
                         const double *suffix_k, const double *suffix_v, double scale,
                         double *dq, double *dk_suffix, double *dv_suffix,
                         int B, int Hq, int Hkv, int S, int P, int d)
{
    return attn_bwd_impl(dout, NULL, q, prefix_k, prefix_v, suffix_k, suffix_v, scale, dq, dk_suffix,
                         dv_suffix, B, Hq, Hkv, S, P, d);
}

/*
 * Backward of L = sum(out * dout) + sum(lse * dlse): the log-sum-exp is a second output of the
 * forward pass, and a caller that uses it (to merge this call's result with another partial
 * attention result, or in a loss) sends a gradient back through it.  Since lse = ln sum_j exp(s_j),
 * d lse / d s_j = p_j, so the only change to the closed form above is ds_j = p_j (dp_j - D + dlse);
 * dV receives nothing from lse.  dlse is [B][Hq][S].
 */
int pskv_oracle_attn_bwd_lse(const double *dout, const double *dlse, const double *q,
                             const double *prefix_k, const double *prefix_v,
                             const double *suffix_k, const double *suffix_v, double scale,
                             double *dq, double *dk_suffix, double *dv_suffix,
                             int B, int Hq, int Hkv, int S, int P, int d)
{
    if (!dlse) return 1;
    return attn_bwd_impl(dout, dlse, q, prefix_k, prefix_v, suffix_k, suffix_v, scale, dq, dk_suffix,
                         dv_suffix, B, Hq, Hkv, S, P, d);
}

/*
 * Batched multi-instruction variant (Sec. 4.3, suffix-centric alignment; appendix on
 * position consistency under padding).  There are Bp prefix caches of padded
 * length Pmax, prefix_k / prefix_v [Bp][Hkv][Pmax][d], and a prefix attention
 * mask m[Bp][Pmax] (1 on real prefix tokens, 0 on padding: "padding tokens are
 * excluded from attention").  Candidate b belongs to instruction b / (B / Bp):
 * each cache is reused by its B / Bp candidates.  The keys a query row sees are
 * the real prefix tokens of its instruction, in order, followed by the
 * candidate's own suffix keys 0..i -- exactly the unpadded sequence.  Here that
 * is written out literally: the masked rows are gathered into a per-candidate
 * K/V copy and ordinary attention (Eq. 2) runs on it.  Any 0/1 mask is
 * accepted, not only left padding.
 */
static int gather_prefix(const double *prefix, const int *mask, double *full, int inst, int g,
                         int Hkv, int Pmax, int d)
{
    int n = 0;
    for (int j = 0; j < Pmax; ++j) {
        if (mask[(size_t)inst * Pmax + j]) {
            memcpy(full + (size_t)n * d, prefix + (((size_t)inst * Hkv + g) * Pmax + j) * d, sizeof(double) * (size_t)d);
            ++n;
        }
    }
    return n;
}

int pskv_oracle_attn_fwd_multi(const double *q, const double *prefix_k, const double *prefix_v,
                               const int *mask, const double *suffix_k, const double *suffix_v,
                               double scale, double *out, double *lse,
                               int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d)
{
    if (B < 1 || Bp < 1 || B % Bp != 0 || Hq < 1 || Hkv < 1 || S < 1 || Pmax < 0 || d < 1 || Hq % Hkv != 0) return 1;
    const int n_rep = Hq / Hkv, Kq = B / Bp;
    const int T = Pmax + S;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int inst = b / Kq;
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        if (!Kf || !Vf || !p) {
            failed = 1;
        } else {
            for (int g = 0; g < Hkv; ++g) {
                const int n = gather_prefix(prefix_k, mask, Kf, inst, g, Hkv, Pmax, d);
                gather_prefix(prefix_v, mask, Vf, inst, g, Hkv, Pmax, d);
                memcpy(Kf + (size_t)n * d, suffix_k + ((size_t)b * Hkv + g) * S * d, sizeof(double) * (size_t)S * d);
                memcpy(Vf + (size_t)n * d, suffix_v + ((size_t)b * Hkv + g) * S * d, sizeof(double) * (size_t)S * d);
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < S; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * S + i;
                        const int n_vis = n + i + 1;
                        lse[row] = softmax_row(q + row * d, Kf, n_vis, d, scale, p);
                        double *o = out + row * d;
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
    }
    return failed ? 2 : 0;
}

/* Backward of the multi-instruction forward: the closed form of pskv_oracle_attn_bwd on the
 * gathered keys; prefix caches are frozen, only dq, dk_suffix, dv_suffix are produced. */
int pskv_oracle_attn_bwd_multi(const double *dout, const double *q, const double *prefix_k,
                               const double *prefix_v, const int *mask, const double *suffix_k,
                               const double *suffix_v, double scale, double *dq, double *dk_suffix,
                               double *dv_suffix, int B, int Bp, int Hq, int Hkv, int S, int Pmax, int d)
{
    if (B < 1 || Bp < 1 || B % Bp != 0 || Hq < 1 || Hkv < 1 || S < 1 || Pmax < 0 || d < 1 || Hq % Hkv != 0) return 1;
    const int n_rep = Hq / Hkv, Kq = B / Bp;
    const int T = Pmax + S;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int inst = b / Kq;
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        if (!Kf || !Vf || !p || !o) {
            failed = 1;
        } else {
            for (int g = 0; g < Hkv; ++g) {
                const int n = gather_prefix(prefix_k, mask, Kf, inst, g, Hkv, Pmax, d);
                gather_prefix(prefix_v, mask, Vf, inst, g, Hkv, Pmax, d);
                memcpy(Kf + (size_t)n * d, suffix_k + ((size_t)b * Hkv + g) * S * d, sizeof(double) * (size_t)S * d);
                memcpy(Vf + (size_t)n * d, suffix_v + ((size_t)b * Hkv + g) * S * d, sizeof(double) * (size_t)S * d);
                double *dKs = dk_suffix + ((size_t)b * Hkv + g) * S * d;
                double *dVs = dv_suffix + ((size_t)b * Hkv + g) * S * d;
                for (size_t e = 0; e < (size_t)S * d; ++e) { dKs[e] = 0.0; dVs[e] = 0.0; }
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < S; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * S + i;
                        const int n_vis = n + i + 1;
                        const double *qr = q + row * d;
                        const double *go = dout + row * d;
                        softmax_row(qr, Kf, n_vis, d, scale, p);
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                        double D = 0.0;
                        for (int c = 0; c < d; ++c) D += go[c] * o[c];
                        double *dqr = dq + row * d;
                        for (int c = 0; c < d; ++c) dqr[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j) {
                            double dp = 0.0;
                            for (int c = 0; c < d; ++c) dp += go[c] * Vf[(size_t)j * d + c];
                            const double ds = p[j] * (dp - D);
                            for (int c = 0; c < d; ++c) dqr[c] += scale * ds * Kf[(size_t)j * d + c];
                            if (j >= n) {
                                const int t = j - n;
                                for (int c = 0; c < d; ++c) {
                                    dKs[(size_t)t * d + c] += scale * ds * qr[c];
                                    dVs[(size_t)t * d + c] += p[j] * go[c];
                                }
                            }
                        }
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
        free(o);
    }
    return failed ? 2 : 0;
}

/*
 * Decode-shaped variant: token-by-token growth of the suffix (the beam-search and
 * sampling-based attacks of the related-work discussion extend every candidate by a few
 * tokens per step on top of what is already cached).  Each candidate b has a suffix cache
 * buffer of Skv rows of which the first len[b] are real (Sq <= len[b] <= Skv; rows past
 * len[b] are ignored whatever they hold), and only the LAST Sq of those len[b] suffix
 * tokens are queries: query i is suffix token len[b] - Sq + i, so by Eq. 2's causal mask
 * it sees the P prefix keys and suffix keys 0 .. len[b] - Sq + i.  With Sq == Skv == len[b]
 * this is pskv_oracle_attn_fwd.  Written out literally: the candidate's real keys are
 * copied behind its own copy of the prefix and each query row runs Eq. 2 on what it sees.
 *
 * Layouts: q, out, dout, dq [B][Hq][Sq][d]; suffix_k, suffix_v, dk_suffix, dv_suffix
 * [B][Hkv][Skv][d]; lse [B][Hq][Sq]; len [B] (NULL = every candidate uses all Skv rows).
 */
static int decode_args_ok(const int *len, int B, int Hq, int Hkv, int Sq, int Skv, int P, int d)
{
    if (B < 1 || Hq < 1 || Hkv < 1 || Sq < 1 || Skv < Sq || P < 0 || d < 1 || Hq % Hkv != 0) return 0;
    if (len)
        for (int b = 0; b < B; ++b)
            if (len[b] < Sq || len[b] > Skv) return 0;
    return 1;
}

int pskv_oracle_attn_fwd_decode(const double *q, const double *prefix_k, const double *prefix_v,
                                const double *suffix_k, const double *suffix_v, const int *len,
                                double scale, double *out, double *lse,
                                int B, int Hq, int Hkv, int Sq, int Skv, int P, int d)
{
    if (!decode_args_ok(len, B, Hq, Hkv, Sq, Skv, P, d)) return 1;
    const int n_rep = Hq / Hkv;
    const int T = P + Skv;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int L = len ? len[b] : Skv;
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        if (!Kf || !Vf || !p) {
            failed = 1;
        } else {
            for (int g = 0; g < Hkv; ++g) {
                memcpy(Kf, prefix_k + (size_t)g * P * d, sizeof(double) * (size_t)P * d);
                memcpy(Vf, prefix_v + (size_t)g * P * d, sizeof(double) * (size_t)P * d);
                memcpy(Kf + (size_t)P * d, suffix_k + ((size_t)b * Hkv + g) * Skv * d, sizeof(double) * (size_t)L * d);
                memcpy(Vf + (size_t)P * d, suffix_v + ((size_t)b * Hkv + g) * Skv * d, sizeof(double) * (size_t)L * d);
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < Sq; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * Sq + i;
                        const int pos = L - Sq + i;          /* suffix position of this query */
                        const int n_vis = P + pos + 1;
                        lse[row] = softmax_row(q + row * d, Kf, n_vis, d, scale, p);
                        double *o = out + row * d;
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
    }
    return failed ? 2 : 0;
}

/* Backward of the decode-shaped forward: the closed form of pskv_oracle_attn_bwd with the
 * shifted causal mask.  Every real suffix key (also those older than the queries) receives a
 * gradient; rows past len[b] of dk_suffix / dv_suffix are zero.  The prefix stays frozen. */
int pskv_oracle_attn_bwd_decode(const double *dout, const double *q, const double *prefix_k,
                                const double *prefix_v, const double *suffix_k, const double *suffix_v,
                                const int *len, double scale, double *dq, double *dk_suffix,
                                double *dv_suffix, int B, int Hq, int Hkv, int Sq, int Skv, int P, int d)
{
    if (!decode_args_ok(len, B, Hq, Hkv, Sq, Skv, P, d)) return 1;
    const int n_rep = Hq / Hkv;
    const int T = P + Skv;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        const int L = len ? len[b] : Skv;
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        if (!Kf || !Vf || !p || !o) {
            failed = 1;
        } else {
            for (int g = 0; g < Hkv; ++g) {
                memcpy(Kf, prefix_k + (size_t)g * P * d, sizeof(double) * (size_t)P * d);
                memcpy(Vf, prefix_v + (size_t)g * P * d, sizeof(double) * (size_t)P * d);
                memcpy(Kf + (size_t)P * d, suffix_k + ((size_t)b * Hkv + g) * Skv * d, sizeof(double) * (size_t)L * d);
                memcpy(Vf + (size_t)P * d, suffix_v + ((size_t)b * Hkv + g) * Skv * d, sizeof(double) * (size_t)L * d);
                double *dKs = dk_suffix + ((size_t)b * Hkv + g) * Skv * d;
                double *dVs = dv_suffix + ((size_t)b * Hkv + g) * Skv * d;
                for (size_t e = 0; e < (size_t)Skv * d; ++e) { dKs[e] = 0.0; dVs[e] = 0.0; }
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < Sq; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * Sq + i;
                        const int n_vis = P + (L - Sq + i) + 1;
                        const double *qr = q + row * d;
                        const double *go = dout + row * d;
                        softmax_row(qr, Kf, n_vis, d, scale, p);
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                        double D = 0.0;
                        for (int c = 0; c < d; ++c) D += go[c] * o[c];
                        double *dqr = dq + row * d;
                        for (int c = 0; c < d; ++c) dqr[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j) {
                            double dp = 0.0;
                            for (int c = 0; c < d; ++c) dp += go[c] * Vf[(size_t)j * d + c];
                            const double ds = p[j] * (dp - D);
                            for (int c = 0; c < d; ++c) dqr[c] += scale * ds * Kf[(size_t)j * d + c];
                            if (j >= P) {
                                const int t = j - P;
                                for (int c = 0; c < d; ++c) {
                                    dKs[(size_t)t * d + c] += scale * ds * qr[c];
                                    dVs[(size_t)t * d + c] += p[j] * go[c];
                                }
                            }
                        }
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
        free(o);
    }
    return failed ? 2 : 0;
}

/*
 * Masked target cross-entropy on top of the vocabulary projection (appendix on the loss:
 * L = sum m^tar CE(logits, z) / sum m^tar, the loss mask being one only on the target-response
 * span).  For N candidates of Lr scored positions each:
 *   logits[r, v] = <hidden[r, :], weight[v, :]>                (the output head, no bias)
 *   lse[r]       = ln sum_v exp(logits[r, v])
 *   nll[r]       = mask[r] * (lse[r] - logits[r, target[r]])   (CE of position r against its token)
 *   loss[c]      = sum_{r in candidate c} nll[r] / sum_{r in c} mask[r]    (0 if the candidate has
 *                  no weighted position): the masked average, per candidate, which is what ranks
 *                  the candidates of one search step; the paper's scalar is the same ratio over all
 *                  candidates and instructions.
 * Written out literally: the full logits row is formed and reduced.  Layouts: hidden [N*Lr][Dm],
 * weight [V][Dm], target [N*Lr] (ints in [0, V) wherever mask != 0), mask [N*Lr].
 */
int pskv_oracle_target_ce_fwd(const double *hidden, const double *weight, const int *target,
                              const double *mask, double *nll, double *lse, double *loss,
                              int N, int Lr, int Dm, int V)
{
    if (N < 1 || Lr < 1 || Dm < 1 || V < 1) return 1;
    const long long R = (long long)N * Lr;
    for (long long r = 0; r < R; ++r)
        if (mask[r] != 0.0 && (target[r] < 0 || target[r] >= V)) return 1;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int c = 0; c < N; ++c) {
        double *z = (double *)malloc(sizeof(double) * (size_t)V);
        if (!z) {
            failed = 1;
        } else {
            double num = 0.0, den = 0.0;
            for (int i = 0; i < Lr; ++i) {
                const long long r = (long long)c * Lr + i;
                const double *h = hidden + r * Dm;
                double m = -INFINITY;
                for (int v = 0; v < V; ++v) {
                    double acc = 0.0;
                    for (int k = 0; k < Dm; ++k) acc += h[k] * weight[(size_t)v * Dm + k];
                    z[v] = acc;
                    if (acc > m) m = acc;
                }
                double l = 0.0;
                for (int v = 0; v < V; ++v) l += exp(z[v] - m);
                lse[r] = m + log(l);
                nll[r] = mask[r] != 0.0 ? mask[r] * (lse[r] - z[target[r]]) : 0.0;
                num += nll[r];
                den += mask[r];
            }
            loss[c] = den != 0.0 ? num / den : 0.0;
        }
        free(z);
    }
    return failed ? 2 : 0;
}

/*
 * Gradients of the shared prefix cache (full differentiability; the search itself keeps the
 * prefix frozen, Sec. 4.2).  The same closed form as pskv_oracle_attn_bwd, keeping what that
 * function discards: for every prefix key j < P of KV head g
 *   dk_prefix[g, j, :] = scale * sum over candidates b, heads h of g, rows i of  ds_j q[b,h,i,:]
 *   dv_prefix[g, j, :] =         sum over the same (b, h, i) of                  p_j dout[b,h,i,:]
 * with ds_j = p_j (dp_j - D + dlse[b,h,i]) (dlse may be NULL).  Because the cache is shared, the sums
 * run over ALL candidates: one KV head per thread, candidates in order, so the result does not
 * depend on the thread count.  dk_prefix, dv_prefix are [Hkv][P][d].
 */
int pskv_oracle_attn_bwd_prefix(const double *dout, const double *dlse, const double *q,
                                const double *prefix_k, const double *prefix_v,
                                const double *suffix_k, const double *suffix_v, double scale,
                                double *dk_prefix, double *dv_prefix,
                                int B, int Hq, int Hkv, int S, int P, int d)
{
    if (B < 1 || Hq < 1 || Hkv < 1 || S < 1 || P < 0 || d < 1 || Hq % Hkv != 0) return 1;
    const int n_rep = Hq / Hkv;
    const int T = P + S;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 1)
    for (int g = 0; g < Hkv; ++g) {
        double *Kf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *Vf = (double *)malloc(sizeof(double) * (size_t)T * d);
        double *p = (double *)malloc(sizeof(double) * (size_t)T);
        double *o = (double *)malloc(sizeof(double) * (size_t)d);
        double *dKp = dk_prefix + (size_t)g * P * d;
        double *dVp = dv_prefix + (size_t)g * P * d;
        for (size_t e = 0; e < (size_t)P * d; ++e) { dKp[e] = 0.0; dVp[e] = 0.0; }
        if (!Kf || !Vf || !p || !o) {
            failed = 1;
        } else {
            for (int b = 0; b < B; ++b) {
                build_full_kv(prefix_k, suffix_k, Kf, b, g, Hkv, S, P, d);
                build_full_kv(prefix_v, suffix_v, Vf, b, g, Hkv, S, P, d);
                for (int r = 0; r < n_rep; ++r) {
                    const int h = g * n_rep + r;
                    for (int i = 0; i < S; ++i) {
                        const size_t row = ((size_t)b * Hq + h) * S + i;
                        const int n_vis = P + i + 1;
                        const double *qr = q + row * d;
                        const double *go = dout + row * d;
                        softmax_row(qr, Kf, n_vis, d, scale, p);
                        for (int c = 0; c < d; ++c) o[c] = 0.0;
                        for (int j = 0; j < n_vis; ++j)
                            for (int c = 0; c < d; ++c) o[c] += p[j] * Vf[(size_t)j * d + c];
                        double D = 0.0;
                        for (int c = 0; c < d; ++c) D += go[c] * o[c];
                        const double gl = dlse ? dlse[row] : 0.0;
                        for (int j = 0; j < P; ++j) {
                            double dp = 0.0;
                            for (int c = 0; c < d; ++c) dp += go[c] * Vf[(size_t)j * d + c];
                            const double ds = p[j] * (dp - D + gl);
                            for (int c = 0; c < d; ++c) {
                                dKp[(size_t)j * d + c] += scale * ds * qr[c];
                                dVp[(size_t)j * d + c] += p[j] * go[c];
                            }
                        }
                    }
                }
            }
        }
        free(Kf);
        free(Vf);
        free(p);
        free(o);
    }
    return failed ? 2 : 0;
}

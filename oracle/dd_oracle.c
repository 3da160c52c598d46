/*
 * dd_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * Plain, slow, fp64 CPU statement of what one DualDiffusion verification step
 * computes: full-sequence bidirectional attention and the verification
 * algorithms (Trust Verifier, KL-divergence remasking, confidence remasking).
 * It exists so that the CUDA library can be compared against something that a
 * reader can check against the paper by eye.  It shares no code, header, table
 * or constant with the CUDA path, is never linked into it, and nothing on the
 * product path may call it: only the tests, the smoke check and the benchmark's
 * CPU-baseline leg do.
 *
 * No tiling, no online softmax, no fusion: every function below is the
 * definition written out with loops.  The only parallelism is an OpenMP
 * "parallel for" over independent rows.
 *
 * Pin status (what fixes each function other than itself is in tests/):
 *   dd_oracle_attention        pinned   (softmax rows sum to 1, constant V,
 *                                        key permutation, N=1, zero keys,
 *                                        one-hot limit, scipy fp64 softmax)
 *   dd_oracle_block_attention  pinned   (numpy fp64 softmax on the valid keys,
 *                                        truncation to kv_len, layout transpose,
 *                                        one key, constant V, zero keys)
 *   dd_oracle_row_scores       pinned   (KL(p,p)=0, KL>=0, two-token closed
 *                                        form, constant logits, shift
 *                                        invariance, scipy rel_entr)
 *   dd_oracle_philox4x32_10    pinned   (published known-answer vectors)
 *   dd_oracle_verify           threshold / probabilistic rules and Trust mode
 *                              pinned (hand-built cases, brute-force argmax,
 *                              Eq. 6 sums to one, empirical frequencies);
 *                              the top-k minimum-keep rule and the choice of
 *                              emitted token at kept positions are readings
 *                              that the paper does not fix: PARITY UNPINNED
 *                              for those two (checked only against a brute
 *                              force restatement of the same reading).
 *   dd_oracle_lm_head          pinned   (identity and one-hot weights, numpy fp64
 *                                        matmul); dd_oracle_verify_f64 is
 *                                        dd_oracle_verify's algorithm on fp64 logits
 *                                        (pinned against it on bf16-exact logits)
 *   dd_oracle_unmask           pinned for the threshold rule and the fixed
 *                              number per step (hand-built cases, scipy
 *                              softmax + numpy argsort on random inputs,
 *                              monotonicity in tau); which of the two rules
 *                              a caller combines, and ties to the lower
 *                              position, are readings: PARITY UNPINNED for
 *                              the tie order.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------ */
/* bf16 -> fp64, exact: a bf16 is the upper 16 bits of an IEEE binary32.     */
static double bf16_to_f64(uint16_t h)
{
    uint32_t w = (uint32_t)h << 16;
    float f;
    memcpy(&f, &w, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------------ */
/* Bidirectional attention, Eq. 3 with the key range equal to the whole
 * sequence (Section 2.2: every token attends to all L positions):
 *     z_i = softmax_j( scale * q_i . k_j ) V ,  j = 0..N-1.
 *
 * q,k,v : [B,H,N,D] bf16 bit patterns, D innermost.
 * rows  : optional list of nrows query indices (the same list is used for
 *         every (b,h)); NULL means all N rows and nrows is ignored.
 * out   : [B,H,R,D] fp64, R = nrows or N.
 * lse   : [B,H,R] fp64, log-sum-exp of the scaled scores of each row; nullable.
 */
void dd_oracle_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                         int B, int H, int N, int D, double scale,
                         const int32_t *rows, int nrows,
                         double *out, double *lse)
{
    const int R = rows ? nrows : N;
    const long total = (long)B * H * R;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)N);
#pragma omp for schedule(dynamic, 16)
        for (long t = 0; t < total; ++t) {
            const long bh = t / R;
            const int r = (int)(t % R);
            const int i = rows ? rows[r] : r;
            const uint16_t *qi = q + ((size_t)bh * N + i) * D;
            const uint16_t *kb = k + (size_t)bh * N * D;
            const uint16_t *vb = v + (size_t)bh * N * D;
            /* scores */
            double m = -INFINITY;
            for (int j = 0; j < N; ++j) {
                double dot = 0.0;
                for (int d = 0; d < D; ++d)
                    dot += bf16_to_f64(qi[d]) * bf16_to_f64(kb[(size_t)j * D + d]);
                s[j] = scale * dot;
                if (s[j] > m) m = s[j];
            }
            /* softmax weights */
            double denom = 0.0;
            for (int j = 0; j < N; ++j) {
                s[j] = exp(s[j] - m);
                denom += s[j];
            }
            /* weighted average of the value rows */
            double *o = out + (size_t)t * D;
            for (int d = 0; d < D; ++d) {
                double acc = 0.0;
                for (int j = 0; j < N; ++j)
                    acc += s[j] * bf16_to_f64(vb[(size_t)j * D + d]);
                o[d] = acc / denom;
            }
            if (lse) lse[t] = m + log(denom);
        }
        free(s);
    }
}

/* The softmax weights of one query row (tests only): p[j], j = 0..N-1. */
void dd_oracle_attention_probs(const uint16_t *q, const uint16_t *k,
                               int H, int N, int D, double scale,
                               int b, int h, int i, double *p)
{
    const size_t bh = (size_t)b * H + h;
    const uint16_t *qi = q + (bh * N + i) * D;
    const uint16_t *kb = k + bh * N * D;
    double m = -INFINITY;
    for (int j = 0; j < N; ++j) {
        double dot = 0.0;
        for (int d = 0; d < D; ++d)
            dot += bf16_to_f64(qi[d]) * bf16_to_f64(kb[(size_t)j * D + d]);
        p[j] = scale * dot;
        if (p[j] > m) m = p[j];
    }
    double denom = 0.0;
    for (int j = 0; j < N; ++j) {
        p[j] = exp(p[j] - m);
        denom += p[j];
    }
    for (int j = 0; j < N; ++j) p[j] /= denom;
}

/* ------------------------------------------------------------------------ */
/* Attention of a block of queries over stored keys and values: Eq. 3 as it is
 * written (queries of the positions being computed, keys and values of the
 * context), the shape of a drafter step with a block-wise KV cache
 * (Section 2.3):
 *     z_i = softmax_{j < n_b}( scale * q_i . k_j ) V ,   i = 0..Nq-1,
 * n_b = kv_len[b] clamped to [0,Nkv] (Nkv if kv_len is NULL); keys at and
 * beyond n_b are padding.  n_b = 0 gives z = 0.
 *
 * head_major = 1: q [B,H,Nq,D], k,v [B,H,Nkv,D]; 0: q [B,Nq,H,D], k,v [B,Nkv,H,D].
 * out: fp64 in the layout of q.                                              */
static size_t elem_index(int head_major, int H, int N, int D, int b, int h, int n, int d)
{
    return head_major ? (((size_t)b * H + h) * N + n) * D + d
                      : (((size_t)b * N + n) * H + h) * D + d;
}

void dd_oracle_block_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                               int B, int H, int Nq, int Nkv, int D,
                               const int32_t *kv_len, int head_major, double scale,
                               double *out)
{
    const long total = (long)B * H * Nq;
#pragma omp parallel
    {
        double *w = (double *)malloc(sizeof(double) * (size_t)Nkv);
#pragma omp for schedule(dynamic, 16)
        for (long t = 0; t < total; ++t) {
            const int b = (int)(t / ((long)H * Nq));
            const int h = (int)((t / Nq) % H);
            const int i = (int)(t % Nq);
            int n = kv_len ? kv_len[b] : Nkv;
            if (n < 0) n = 0;
            if (n > Nkv) n = Nkv;
            double m = -INFINITY;
            for (int j = 0; j < n; ++j) {
                double dot = 0.0;
                for (int d = 0; d < D; ++d)
                    dot += bf16_to_f64(q[elem_index(head_major, H, Nq, D, b, h, i, d)]) *
                           bf16_to_f64(k[elem_index(head_major, H, Nkv, D, b, h, j, d)]);
                w[j] = scale * dot;
                if (w[j] > m) m = w[j];
            }
            double denom = 0.0;
            for (int j = 0; j < n; ++j) {
                w[j] = exp(w[j] - m);
                denom += w[j];
            }
            for (int d = 0; d < D; ++d) {
                double acc = 0.0;
                for (int j = 0; j < n; ++j)
                    acc += w[j] * bf16_to_f64(v[elem_index(head_major, H, Nkv, D, b, h, j, d)]);
                out[elem_index(head_major, H, Nq, D, b, h, i, d)] = n > 0 ? acc / denom : 0.0;
            }
        }
        free(w);
    }
}

/* ------------------------------------------------------------------------ */
/* Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as
 * easy as 1, 2, 3", SC'11).  Ten rounds; the key is bumped by the Weyl
 * constants between rounds.                                                 */
void dd_oracle_philox4x32_10(const uint32_t ctr_in[4], const uint32_t key_in[2],
                             uint32_t out[4])
{
    uint32_t c0 = ctr_in[0], c1 = ctr_in[1], c2 = ctr_in[2], c3 = ctr_in[3];
    uint32_t k0 = key_in[0], k1 = key_in[1];
    for (int round = 0; round < 10; ++round) {
        const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        const uint32_t n1 = (uint32_t)p1;
        const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        const uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* The uniform u in [0,1) drawn for position i of sequence b: key = the two
 * halves of the seed, counter = (i, b, 0, 0), first output word, top 24 bits.
 * A multiple of 2^-24 is exact in both fp32 and fp64.                       */
double dd_oracle_uniform(uint64_t seed, int b, int i)
{
    const uint32_t ctr[4] = {(uint32_t)i, (uint32_t)b, 0u, 0u};
    const uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32)};
    uint32_t r[4];
    dd_oracle_philox4x32_10(ctr, key, r);
    return (double)(r[0] >> 8) * (1.0 / 16777216.0);
}

/* ------------------------------------------------------------------------ */
/* Per-position quantities of Section 3.2 for one pair of logit rows.
 *   argmax_v : verifier's most likely token, lowest index among exact ties
 *   conf     : c_V = max_x p_V(x)                                   (Eq. 7)
 *   kl       : KL(p_D || p_V) = sum_x p_D(x) (ln p_D(x) - ln p_V(x)) (Eq. 5),
 *              natural log, clamped at zero; 0 if drafter row is NULL.
 */
static void row_scores_f64(const double *drafter_row, const double *verifier_row,
                           int V, int32_t *argmax_v, double *conf, double *kl)
{
    /* verifier: argmax and log-softmax */
    int a = 0;
    double mv = verifier_row[0];
    for (int x = 1; x < V; ++x) {
        const double l = verifier_row[x];
        if (l > mv) { mv = l; a = x; }
    }
    double zv = 0.0;
    for (int x = 0; x < V; ++x) zv += exp(verifier_row[x] - mv);
    const double lse_v = mv + log(zv);
    *argmax_v = a;
    *conf = exp(mv - lse_v);

    double acc = 0.0;
    if (drafter_row) {
        double md = -INFINITY;
        for (int x = 0; x < V; ++x) {
            const double l = drafter_row[x];
            if (l > md) md = l;
        }
        double zd = 0.0;
        for (int x = 0; x < V; ++x) zd += exp(drafter_row[x] - md);
        const double lse_d = md + log(zd);
        for (int x = 0; x < V; ++x) {
            const double log_pd = drafter_row[x] - lse_d;
            const double log_pv = verifier_row[x] - lse_v;
            /* a token the drafter excludes (logit -inf, p_D(x) = 0) adds nothing: the
             * Kullback-Leibler sum of Eq. 5 runs over the support of p_D (0 ln 0 = 0) */
            if (log_pd == -INFINITY) continue;
            acc += exp(log_pd) * (log_pd - log_pv);
        }
        if (acc < 0.0) acc = 0.0;
    }
    *kl = acc;
}

/* The same for rows stored as bf16: converted exactly, then the arithmetic above. */
void dd_oracle_row_scores(const uint16_t *drafter_row, const uint16_t *verifier_row,
                          int V, int32_t *argmax_v, double *conf, double *kl)
{
    double *v = (double *)malloc(sizeof(double) * (size_t)V);
    double *d = drafter_row ? (double *)malloc(sizeof(double) * (size_t)V) : NULL;
    for (int x = 0; x < V; ++x) {
        v[x] = bf16_to_f64(verifier_row[x]);
        if (d) d[x] = bf16_to_f64(drafter_row[x]);
    }
    row_scores_f64(d, v, V, argmax_v, conf, kl);
    free(v);
    free(d);
}

/* ------------------------------------------------------------------------ */
enum { MODE_TRUST = 0, MODE_KL = 1, MODE_CONF = 2 };
enum { FLAG_PROBABILISTIC = 0x100, FLAG_EMIT_DRAFTER = 0x200 };

#define EXEMPT_BAND 1e-5

/* Verification algorithm A(p_D, p_V, x^D) of Algorithm 1, Section 3.2.
 *
 * drafter, verifier : [B,P,V] bf16 bit patterns (drafter may be NULL unless
 *                     mode is KL)
 * tokens            : [B,P] current ids x^D
 * flags             : [B,P] 1 = position belongs to the drafter-decoded set
 * mode              : low 8 bits TRUST/KL/CONF, plus FLAG_* bits
 * tau, k, seed      : threshold, minimum-keep count, Philox seed
 * out_tokens [B,P], out_mask [B,P] (1 = remasked), out_score [B,P] fp64,
 * exempt [B,P] (1 = decision lies within 1e-5 of a boundary; nullable)
 *
 * Returns 0, or -1 on an unknown mode.
 */
static int verify_core(const uint16_t *drafter, const uint16_t *verifier,
                       const double *drafter_f64, const double *verifier_f64,
                       const int32_t *tokens, const uint8_t *flags,
                       int mode, double tau, int k, uint64_t seed,
                       int32_t *out_tokens, uint8_t *out_mask, double *out_score,
                       uint8_t *exempt, int B, int P, int V)
{
    const int algo = mode & 0xFF;
    const int probabilistic = (mode & FLAG_PROBABILISTIC) != 0;
    const int emit_drafter = (mode & FLAG_EMIT_DRAFTER) != 0;
    if (algo != MODE_TRUST && algo != MODE_KL && algo != MODE_CONF) return -1;
    if (algo == MODE_KL && !drafter && !drafter_f64) return -1;

    const long BP = (long)B * P;
    int32_t *amax = (int32_t *)malloc(sizeof(int32_t) * (size_t)BP);
    double *conf = (double *)malloc(sizeof(double) * (size_t)BP);
    double *kl = (double *)malloc(sizeof(double) * (size_t)BP);

    /* Step 1-2: per-position argmax, confidence, KL (flagged positions only) */
#pragma omp parallel for schedule(dynamic, 1)
    for (long t = 0; t < BP; ++t) {
        amax[t] = 0; conf[t] = 0.0; kl[t] = 0.0;
        if (!flags[t]) continue;
        if (verifier_f64) {      /* logits handed over in fp64 (the fused language-model head) */
            const double *dd = (algo == MODE_KL) ? drafter_f64 + (size_t)t * V : NULL;
            row_scores_f64(dd, verifier_f64 + (size_t)t * V, V, &amax[t], &conf[t], &kl[t]);
        } else {
            const uint16_t *dv = verifier + (size_t)t * V;
            const uint16_t *dd = (algo == MODE_KL) ? drafter + (size_t)t * V : NULL;
            dd_oracle_row_scores(dd, dv, V, &amax[t], &conf[t], &kl[t]);
        }
    }

    int *members = (int *)malloc(sizeof(int) * (size_t)P);
    double *rel = (double *)malloc(sizeof(double) * (size_t)P);
    int *rank = (int *)malloc(sizeof(int) * (size_t)P);

    for (int b = 0; b < B; ++b) {
        const long base = (long)b * P;
        /* the drafter-decoded set of this sequence */
        int n = 0;
        for (int i = 0; i < P; ++i)
            if (flags[base + i]) members[n++] = i;

        /* Eq. 6 denominator */
        double kl_sum = 0.0;
        for (int a = 0; a < n; ++a) kl_sum += kl[base + members[a]];

        /* Step 4 preparation: reliability and its rank (0 = most reliable);
         * ties go to the lower position.                                    */
        for (int a = 0; a < n; ++a) {
            const int i = members[a];
            rel[a] = (algo == MODE_KL) ? -kl[base + i] : conf[base + i];
        }
        for (int a = 0; a < n; ++a) {
            int better = 0;
            for (int c = 0; c < n; ++c) {
                if (c == a) continue;
                if (rel[c] > rel[a] || (rel[c] == rel[a] && members[c] < members[a]))
                    ++better;
            }
            rank[a] = better;
        }
        /* reliabilities just inside and just outside the top-k boundary */
        double r_last_in = NAN, r_first_out = NAN;
        if (k > 0 && k < n) {            /* otherwise no boundary exists */
            for (int a = 0; a < n; ++a) {
                if (rank[a] == k - 1) r_last_in = rel[a];
                if (rank[a] == k) r_first_out = rel[a];
            }
        }

        for (int i = 0; i < P; ++i) {
            out_tokens[base + i] = tokens[base + i];
            out_mask[base + i] = 0;
            out_score[base + i] = 0.0;
            if (exempt) exempt[base + i] = 0;
        }

        for (int a = 0; a < n; ++a) {
            const int i = members[a];
            const long t = base + i;
            int fail = 0, near = 0;
            double score = conf[t];
            if (algo == MODE_KL) {
                score = kl[t];
                if (!probabilistic) {
                    fail = kl[t] > tau;                           /* threshold rule */
                    near = fabs(kl[t] - tau) <= EXEMPT_BAND;
                } else {
                    const double pi = kl_sum > 0.0 ? kl[t] / kl_sum : 0.0; /* Eq. 6 */
                    const double u = dd_oracle_uniform(seed, b, i);
                    fail = u < pi;
                    near = fabs(u - pi) <= EXEMPT_BAND;
                }
            } else if (algo == MODE_CONF) {
                if (!probabilistic) {
                    fail = conf[t] < tau;
                    near = fabs(conf[t] - tau) <= EXEMPT_BAND;
                } else {
                    const double u = dd_oracle_uniform(seed, b, i);
                    fail = u < 1.0 - conf[t];
                    near = fabs(u - (1.0 - conf[t])) <= EXEMPT_BAND;
                }
            }
            /* Step 4: the k most reliable positions are kept whatever Step 3 said */
            const int in_topk = rank[a] < k;
            /* the top-k rule decides a failing position; its place relative to the boundary is
             * uncertain only if the reliability on the other side of the boundary is within the band */
            if (fail) {
                if (in_topk && !isnan(r_first_out) && fabs(rel[a] - r_first_out) <= EXEMPT_BAND) near = 1;
                if (!in_topk && !isnan(r_last_in) && fabs(rel[a] - r_last_in) <= EXEMPT_BAND) near = 1;
            }
            const int remask = fail && !in_topk;
            /* Step 5 */
            out_mask[t] = (uint8_t)remask;
            if (remask || emit_drafter) out_tokens[t] = tokens[t];
            else out_tokens[t] = amax[t];
            out_score[t] = score;
            if (exempt) exempt[t] = (uint8_t)(near && algo != MODE_TRUST);
        }
    }
    free(members); free(rel); free(rank);
    free(amax); free(conf); free(kl);
    return 0;
}

int dd_oracle_verify(const uint16_t *drafter, const uint16_t *verifier,
                     const int32_t *tokens, const uint8_t *flags,
                     int mode, double tau, int k, uint64_t seed,
                     int32_t *out_tokens, uint8_t *out_mask, double *out_score,
                     uint8_t *exempt, int B, int P, int V)
{
    return verify_core(drafter, verifier, NULL, NULL, tokens, flags, mode, tau, k, seed,
                       out_tokens, out_mask, out_score, exempt, B, P, V);
}

/* The same algorithm on logits given in fp64, [B,P,V] (drafter may be NULL unless the mode is KL). */
int dd_oracle_verify_f64(const double *drafter, const double *verifier,
                         const int32_t *tokens, const uint8_t *flags,
                         int mode, double tau, int k, uint64_t seed,
                         int32_t *out_tokens, uint8_t *out_mask, double *out_score,
                         uint8_t *exempt, int B, int P, int V)
{
    if (!verifier) return -1;
    return verify_core(NULL, NULL, drafter, verifier, tokens, flags, mode, tau, k, seed,
                       out_tokens, out_mask, out_score, exempt, B, P, V);
}

/* ------------------------------------------------------------------------ */
/* The language-model head of the verification phase: Algorithm 1 computes p_V(. | x^D) "for all
 * positions", i.e. logits[t, x] = sum_k hidden[t, k] * weight[x, k] (the last hidden state of
 * position t against the output embedding of token x), softmax over x.  hidden [rows, K] and weight
 * [V, K] are bf16 bit patterns; the sum is taken in fp64, in index order.  Rows whose flag is 0 are
 * skipped (left at 0) when flags is not NULL.                                                      */
void dd_oracle_lm_head(const uint16_t *hidden, const uint16_t *weight, const uint8_t *flags,
                       int rows, int K, int V, double *logits)
{
#pragma omp parallel for collapse(2) schedule(static)
    for (int t = 0; t < rows; ++t) {
        for (int x = 0; x < V; ++x) {
            double acc = 0.0;
            if (!flags || flags[t]) {
                const uint16_t *h = hidden + (size_t)t * K, *w = weight + (size_t)x * K;
                for (int j = 0; j < K; ++j) acc += bf16_to_f64(h[j]) * bf16_to_f64(w[j]);
            }
            logits[(size_t)t * V + x] = acc;
        }
    }
}

/* ------------------------------------------------------------------------ */
/* Unmask(p, x): one confidence-based unmasking step of a masked diffusion
 * model (Algorithm 1, drafting phase; Section 2.1: each step reveals the
 * masked positions the model is most sure of; Section 2.3: every position
 * above a confidence threshold, rather than a fixed number per step).
 *
 * For every masked position i (flags = 1): p_i = softmax(logits_i),
 * a_i = argmax (lowest index), c_i = p_i(a_i).  Position i is unmasked iff
 * c_i >= tau, or it is one of the k most confident masked positions of its
 * sequence (ties to the lower position).  tau = +inf gives "a fixed number k
 * per step"; k = 1 guarantees progress under a threshold.
 *
 * out_tokens = a_i where unmasked, tokens[i] otherwise; out_mask = 1 where the
 * position stays masked; out_conf = c_i (0 at positions that were not masked);
 * exempt (nullable) = 1 where the decision lies within 1e-5 of the threshold,
 * or where the count rule decides and the confidence just across the top-k
 * boundary is within 1e-5.                                                   */
typedef struct { double c; int pos; } conf_pos;

static int more_confident_first(const void *x, const void *y)
{
    const conf_pos *a = (const conf_pos *)x, *b = (const conf_pos *)y;
    if (a->c > b->c) return -1;
    if (a->c < b->c) return 1;
    return a->pos < b->pos ? -1 : (a->pos > b->pos ? 1 : 0);
}

void dd_oracle_unmask(const uint16_t *logits, const int32_t *tokens, const uint8_t *flags,
                      double tau, int k,
                      int32_t *out_tokens, uint8_t *out_mask, double *out_conf, uint8_t *exempt,
                      int B, int P, int V)
{
    const long BP = (long)B * P;
    int32_t *best = (int32_t *)malloc(sizeof(int32_t) * (size_t)BP);
#pragma omp parallel for schedule(dynamic, 1)
    for (long t = 0; t < BP; ++t) {
        best[t] = 0;
        out_conf[t] = 0.0;
        if (!flags[t]) continue;
        const uint16_t *row = logits + (size_t)t * V;
        double top = -INFINITY;
        int where = 0;
        for (int x = 0; x < V; ++x) {
            const double l = bf16_to_f64(row[x]);
            if (l > top) { top = l; where = x; }
        }
        double denom = 0.0;
        for (int x = 0; x < V; ++x) denom += exp(bf16_to_f64(row[x]) - top);
        best[t] = where;
        out_conf[t] = 1.0 / denom;           /* exp(top - top) / denom */
    }
    conf_pos *order = (conf_pos *)malloc(sizeof(conf_pos) * (size_t)P);
    for (int b = 0; b < B; ++b) {
        const long base = (long)b * P;
        int n = 0;
        for (int i = 0; i < P; ++i) {
            out_tokens[base + i] = tokens[base + i];
            out_mask[base + i] = 0;
            if (exempt) exempt[base + i] = 0;
            if (flags[base + i]) { order[n].c = out_conf[base + i]; order[n].pos = i; ++n; }
        }
        qsort(order, (size_t)n, sizeof(conf_pos), more_confident_first);
        for (int r = 0; r < n; ++r) {
            const long t = base + order[r].pos;
            const int above = order[r].c >= tau;
            const int unmask = above || r < k;
            out_mask[t] = (uint8_t)!unmask;
            if (unmask) out_tokens[t] = best[t];
            if (exempt) {
                int near = fabs(order[r].c - tau) <= EXEMPT_BAND;
                if (!above && k > 0 && k < n) {      /* the top-k boundary decides: uncertain only if
                                                        the confidence across the boundary is within the band */
                    if (r < k && fabs(order[r].c - order[k].c) <= EXEMPT_BAND) near = 1;
                    if (r >= k && fabs(order[r].c - order[k - 1].c) <= EXEMPT_BAND) near = 1;
                }
                exempt[t] = (uint8_t)near;
            }
        }
    }
    free(order);
    free(best);
}

/* Number of OpenMP threads a parallel region will use (reported by the bench). */
#ifdef _OPENMP
#include <omp.h>
int dd_oracle_threads(void) { return omp_get_max_threads(); }
#else
int dd_oracle_threads(void) { return 1; }
#endif

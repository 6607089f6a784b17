/*
 * CPU oracle for the LVSpec verify step.  TEST INFRASTRUCTURE ONLY: tests, the
 * smoke check and the benchmark's CPU-baseline leg may call it; the product
 * path never does, and it shares no code with the CUDA sources.
 *
 * Everything is written out as the plain definition, in fp64, with no tiling,
 * no online softmax and no reordering, so it can be checked against the paper
 * by eye.  OpenMP only distributes independent (batch, query, head) units and
 * independent logits rows over the host cores.
 *
 * Pinned by tests/test_oracle_*.py against: torch's scaled-dot-product
 * attention in fp64 (the attention the paper names in App. "Baseline
 * Details"), closed forms (identical keys, dominant key, key translation),
 * brute-force enumeration and hand-worked cases of the rule (tests/golden),
 * the closed form of Prop. 2.2, and for the fp8 cache the published E4M3
 * format through an independent library decoder.  The paper prints no worked numeric
 * example of the rule, so beyond those pins the rule is "parity unpinned"
 * against the authors' own code.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

static double bf16_to_double(uint16_t bits)
{
    uint32_t u = ((uint32_t)bits) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/*
 * Verification attention of the gamma draft queries over the cache (Eq. 1: the
 * target model verifies the K draft tokens in one parallel pass; the attention
 * is scaled-dot-product attention, App. "Baseline Details"), plus the visual
 * mass: the share of each query's softmax that lands on the visual span.
 *
 *   q         bf16 bits [B, gamma, Hq, D]
 *   k, v      bf16 bits [B, Hkv, Lmax, D]
 *   kv_len    [B]   cache length including the gamma draft slots (the last ones)
 *   span      [B,2] visual positions [start, end)
 *   out       fp64 [B, gamma, Hq, D]
 *   mass      fp64 [B, gamma, Hq]
 *   probs     optional fp64 [B, gamma, Hq, Lmax] (0 beyond the visible prefix)
 *
 * Query g of a sequence sees positions j < kv_len - gamma + g + 1 (causal over
 * the draft tail).  Head h reads KV head h / (Hq / Hkv).
 *
 * Draft-token trees (App. "Exploration on Draft Token Trees": a static tree of
 * branches with K draft tokens each, every branch verified on its own): the
 * gamma = R * branch_len draft slots at the end of the cache hold the branches
 * one after the other, and query g (branch g / branch_len) sees the context
 * before the draft slots plus the slots of its own branch up to itself.
 * branch_len = gamma is the plain chain above.
 */
void lvspec_oracle_verify_attention_tree(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                         const int32_t *kv_len, const int32_t *span,
                                         int B, int gamma, int branch_len, int Hq, int Hkv, int D,
                                         int Lmax, double *out, double *mass, double *probs);

void lvspec_oracle_verify_attention(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                    const int32_t *kv_len, const int32_t *span,
                                    int B, int gamma, int Hq, int Hkv, int D, int Lmax,
                                    double *out, double *mass, double *probs)
{
    lvspec_oracle_verify_attention_tree(q, k, v, kv_len, span, B, gamma, gamma, Hq, Hkv, D, Lmax, out,
                                        mass, probs);
}

void lvspec_oracle_verify_attention_tree(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                         const int32_t *kv_len, const int32_t *span,
                                         int B, int gamma, int branch_len, int Hq, int Hkv, int D,
                                         int Lmax, double *out, double *mass, double *probs)
{
    const int G = Hq / Hkv;
    const double scale = 1.0 / sqrt((double)D);
    const long units = (long)B * gamma * Hq;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(Lmax > 0 ? Lmax : 1));
        double *qd = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            const int h = (int)(u % Hq);
            const int g = (int)((u / Hq) % gamma);
            const int b = (int)(u / ((long)Hq * gamma));
            const int kvh = h / G;
            const int ctx_len = kv_len[b] - gamma;              /* positions before the draft slots */
            const int own0 = ctx_len + (g / branch_len) * branch_len;   /* first slot of g's branch */
            const int vis = kv_len[b] - gamma + g + 1;          /* one past g's own slot */
            const int vs = span[2 * b], ve = span[2 * b + 1];
            const uint16_t *qrow = q + (((size_t)b * gamma + g) * Hq + h) * D;
            const uint16_t *kb = k + ((size_t)b * Hkv + kvh) * (size_t)Lmax * D;
            const uint16_t *vb = v + ((size_t)b * Hkv + kvh) * (size_t)Lmax * D;
            double *orow = out + (((size_t)b * gamma + g) * Hq + h) * D;

            for (int d = 0; d < D; ++d) qd[d] = bf16_to_double(qrow[d]);
            double m = -INFINITY;
            for (int j = 0; j < vis; ++j) {
                if (j >= ctx_len && j < own0) { s[j] = -INFINITY; continue; }   /* another branch */
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += qd[d] * bf16_to_double(kb[(size_t)j * D + d]);
                s[j] = acc * scale;
                if (s[j] > m) m = s[j];
            }
            double Z = 0.0;
            for (int j = 0; j < vis; ++j) { s[j] = (s[j] == -INFINITY) ? 0.0 : exp(s[j] - m); Z += s[j]; }
            for (int d = 0; d < D; ++d) orow[d] = 0.0;
            double vm = 0.0;
            for (int j = 0; j < vis; ++j) {
                const double p = s[j] / Z;
                if (j >= vs && j < ve) vm += p;
                if (p != 0.0)
                    for (int d = 0; d < D; ++d) orow[d] += p * bf16_to_double(vb[(size_t)j * D + d]);
                if (probs) probs[(((size_t)b * gamma + g) * Hq + h) * (size_t)Lmax + j] = p;
            }
            if (probs)
                for (int j = vis > 0 ? vis : 0; j < Lmax; ++j)
                    probs[(((size_t)b * gamma + g) * Hq + h) * (size_t)Lmax + j] = 0.0;
            mass[((size_t)b * gamma + g) * Hq + h] = vm;
        }
        free(s);
        free(qd);
    }
}

/*
 * An fp8 cache.  The paper's premise is that the target's pass over the long visual
 * KV cache is bound by memory traffic (Sec. 1; the T_t^K term of the speed-up formula in
 * Sec. 2.2); storing K and V in 8 bits halves that traffic.  The stored format is the
 * OCP 8-bit floating point E4M3 ("FN" variant: no infinities): 1 sign bit, 4 exponent
 * bits with bias 7, 3 mantissa bits;
 *     exponent field 0:      value = (-1)^s * 2^-6 * (mantissa / 8)            (subnormal)
 *     otherwise:             value = (-1)^s * 2^(exponent - 7) * (1 + mantissa / 8)
 *     exponent 15 with mantissa 7 (codes 0x7F, 0xFF) is NaN; the largest finite value is 448.
 * A cache element is code * scale, with one fp32 scale per (sequence, KV head) for K and
 * one for V.
 */
double lvspec_oracle_e4m3_decode(uint8_t code)
{
    const int sign = code >> 7, e = (code >> 3) & 15, m = code & 7;
    double x;
    if (e == 15 && m == 7) return NAN;
    if (e == 0) x = ldexp((double)m / 8.0, -6);
    else x = ldexp(1.0 + (double)m / 8.0, e - 7);
    return sign ? -x : x;
}

/*
 * Verification attention with visual mass (Eq. 1; SDPA, App. "Baseline Details") over an
 * fp8 cache: the plain definition of lvspec_oracle_verify_attention_tree, with every
 * cache element decoded as above and multiplied by its scale in fp64 first.
 *
 *   q           bf16 bits [B, gamma, Hq, D]
 *   k8, v8      E4M3 codes [B, Hkv, Lmax, D]
 *   k_scale, v_scale   fp32 [B, Hkv]
 * everything else as for the bf16 cache.
 */
void lvspec_oracle_verify_attention_fp8(const uint16_t *q, const uint8_t *k8, const uint8_t *v8,
                                        const float *k_scale, const float *v_scale,
                                        const int32_t *kv_len, const int32_t *span,
                                        int B, int gamma, int Hq, int Hkv, int D, int Lmax,
                                        double *out, double *mass)
{
    const int G = Hq / Hkv;
    const double scale = 1.0 / sqrt((double)D);
    const long units = (long)B * gamma * Hq;
#pragma omp parallel
    {
        double *s = (double *)malloc(sizeof(double) * (size_t)(Lmax > 0 ? Lmax : 1));
        double *qd = (double *)malloc(sizeof(double) * (size_t)D);
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            const int h = (int)(u % Hq);
            const int g = (int)((u / Hq) % gamma);
            const int b = (int)(u / ((long)Hq * gamma));
            const int kvh = h / G;
            const int vis = kv_len[b] - gamma + g + 1;
            const int vs = span[2 * b], ve = span[2 * b + 1];
            const double ks = (double)k_scale[(size_t)b * Hkv + kvh];
            const double vsc = (double)v_scale[(size_t)b * Hkv + kvh];
            const uint16_t *qrow = q + (((size_t)b * gamma + g) * Hq + h) * D;
            const uint8_t *kb = k8 + ((size_t)b * Hkv + kvh) * (size_t)Lmax * D;
            const uint8_t *vb = v8 + ((size_t)b * Hkv + kvh) * (size_t)Lmax * D;
            double *orow = out + (((size_t)b * gamma + g) * Hq + h) * D;

            for (int d = 0; d < D; ++d) qd[d] = bf16_to_double(qrow[d]);
            double m = -INFINITY;
            for (int j = 0; j < vis; ++j) {
                double acc = 0.0;
                for (int d = 0; d < D; ++d) acc += qd[d] * (lvspec_oracle_e4m3_decode(kb[(size_t)j * D + d]) * ks);
                s[j] = acc * scale;
                if (s[j] > m) m = s[j];
            }
            double Z = 0.0;
            for (int j = 0; j < vis; ++j) { s[j] = exp(s[j] - m); Z += s[j]; }
            for (int d = 0; d < D; ++d) orow[d] = 0.0;
            double vm = 0.0;
            for (int j = 0; j < vis; ++j) {
                const double p = s[j] / Z;
                if (j >= vs && j < ve) vm += p;
                if (p != 0.0)
                    for (int d = 0; d < D; ++d)
                        orow[d] += p * (lvspec_oracle_e4m3_decode(vb[(size_t)j * D + d]) * vsc);
            }
            mass[((size_t)b * gamma + g) * Hq + h] = vm;
        }
        free(s);
        free(qd);
    }
}

/* Ordering used for the loosened set: score ascending, then position ascending
 * (a stable ascending argsort). */
typedef struct { double score; int pos; } scored_t;
static int cmp_scored(const void *a, const void *b)
{
    const scored_t *x = (const scored_t *)a, *y = (const scored_t *)b;
    if (x->score < y->score) return -1;
    if (x->score > y->score) return 1;
    return (x->pos > y->pos) - (x->pos < y->pos);
}

/*
 * Loose acceptance pass (Sec. 3.2 and 3.3).
 *
 *   logits   fp32 [B, gamma, V]   target logits, row i judges draft token i
 *   draft    int32 [B, gamma]
 *   mass     fp32 [B, gamma, Hm]  per-head relevance; Hm = 1 takes a ready score
 *   n_loose  number of loosened positions (the "lambda K lowest" of Eq. 5)
 *   window   shift tolerance W: 0 switches PST off, W >= gamma - 1 is Eq. 7
 *   accept_len int32 [B]; target int32 [B,gamma] and acc uint8 [B,gamma] optional
 *
 * Steps, in the paper's order:
 *  1. y_i = the target's token at position i: the largest logit, first
 *     occurrence on ties; NaN counts as -inf; a row with nothing above -inf
 *     gives token 0.
 *  2. score_i = sum over heads of mass (added in index order, in double).
 *  3. I' = the first n_loose positions of the ascending stable argsort (Eq. 5).
 *  4. nabla_i = 1 if draft_i == y_i; else 1 if i in I'; else 1 if y_i equals a
 *     draft token at a position within W of i; else 0 (Eq. 6 / Eq. 7).
 *  5. accepted length = sum_k prod_{j<=k} nabla_j (Eq. 2).
 */
void lvspec_oracle_loose_accept(const float *logits, const int32_t *draft, const float *mass,
                                int B, int gamma, int V, int Hm, int n_loose, int window,
                                int32_t *accept_len, int32_t *target, uint8_t *acc)
{
#pragma omp parallel for schedule(dynamic, 1)
    for (int b = 0; b < B; ++b) {
        int32_t *y = (int32_t *)malloc(sizeof(int32_t) * (size_t)(gamma > 0 ? gamma : 1));
        uint8_t *nabla = (uint8_t *)malloc((size_t)(gamma > 0 ? gamma : 1));
        uint8_t *loosened = (uint8_t *)calloc((size_t)(gamma > 0 ? gamma : 1), 1);
        scored_t *order = (scored_t *)malloc(sizeof(scored_t) * (size_t)(gamma > 0 ? gamma : 1));

        for (int i = 0; i < gamma; ++i) {
            const float *row = logits + ((size_t)b * gamma + i) * (size_t)V;
            float best = -INFINITY;
            int arg = 0;
            for (int t = 0; t < V; ++t) {
                const float x = row[t];
                if (x > best) { best = x; arg = t; }   /* NaN never wins; first max kept */
            }
            y[i] = arg;
        }
        for (int i = 0; i < gamma; ++i) {
            double sc = 0.0;
            for (int h = 0; h < Hm; ++h) sc += (double)mass[((size_t)b * gamma + i) * Hm + h];
            order[i].score = sc;
            order[i].pos = i;
        }
        qsort(order, (size_t)gamma, sizeof(scored_t), cmp_scored);
        for (int r = 0; r < gamma && r < n_loose; ++r) loosened[order[r].pos] = 1;

        for (int i = 0; i < gamma; ++i) {
            const int32_t *dr = draft + (size_t)b * gamma;
            int ok = (dr[i] == y[i]);
            if (!ok && loosened[i]) ok = 1;
            if (!ok) {
                for (int kk = 0; kk < gamma; ++kk) {
                    const int dist = kk > i ? kk - i : i - kk;
                    if (dist <= window && dr[kk] == y[i]) { ok = 1; break; }
                }
            }
            nabla[i] = (uint8_t)ok;
        }
        int tau = 0;
        for (int kk = 0; kk < gamma; ++kk) {
            int prod = 1;
            for (int j = 0; j <= kk; ++j) prod *= nabla[j];
            tau += prod;
        }
        accept_len[b] = tau;
        if (target) memcpy(target + (size_t)b * gamma, y, sizeof(int32_t) * (size_t)gamma);
        if (acc) memcpy(acc + (size_t)b * gamma, nabla, (size_t)gamma);
        free(y); free(nabla); free(loosened); free(order);
    }
}

/* Number of loosened positions for a loose parameter lambda (Sec. 3.2: "the
 * lambda K tokens with the lowest scores"; the slice 0:lambda K of Eq. 5).  A
 * non-integer product is cut down to the integer below; 1e-9 guards products
 * that land a rounding error under an integer. */
int lvspec_oracle_n_loose(double lambda, int gamma)
{
    return (int)floor(lambda * (double)gamma + 1e-9);
}

/*
 * Visual relevance of the draft tokens as the paper defines it (Sec. 3.1,
 * Eq. 4): the cosine similarity between the final-layer hidden state of each
 * draft token and that of every visual token, then the mean of the N largest
 * similarities along the visual dimension.
 *
 *   h_draft   bf16 bits [B, K, d]     H_D^s of Eq. 3
 *   h_visual  bf16 bits [B, lv, d]    H_V of Eq. 3
 *   top_n     N of Eq. 4 (the paper runs N = 10); min(N, lv) values are averaged
 *   relevance fp64 [B, K]             A_s
 *   cosines   optional fp64 [B, K, lv]
 *
 * A zero vector has no direction: its cosine with anything is taken as 0 (the
 * paper does not meet the case).
 */
static int cmp_desc(const void *a, const void *b)
{
    const double x = *(const double *)a, y = *(const double *)b;
    return (x < y) - (x > y);
}

void lvspec_oracle_visual_relevance(const uint16_t *h_draft, const uint16_t *h_visual,
                                    int B, int K, int lv, int d, int top_n,
                                    double *relevance, double *cosines)
{
    const long units = (long)B * K;
#pragma omp parallel
    {
        double *c = (double *)malloc(sizeof(double) * (size_t)(lv > 0 ? lv : 1));
        double *hd = (double *)malloc(sizeof(double) * (size_t)d);
#pragma omp for schedule(dynamic, 1)
        for (long u = 0; u < units; ++u) {
            const int b = (int)(u / K), k = (int)(u % K);
            const uint16_t *drow = h_draft + ((size_t)b * K + k) * d;
            double nd = 0.0;
            for (int t = 0; t < d; ++t) { hd[t] = bf16_to_double(drow[t]); nd += hd[t] * hd[t]; }
            nd = sqrt(nd);
            for (int j = 0; j < lv; ++j) {
                const uint16_t *vrow = h_visual + ((size_t)b * lv + j) * d;
                double dot = 0.0, nv = 0.0;
                for (int t = 0; t < d; ++t) {
                    const double x = bf16_to_double(vrow[t]);
                    dot += hd[t] * x;
                    nv += x * x;
                }
                nv = sqrt(nv);
                c[j] = (nd > 0.0 && nv > 0.0) ? dot / (nd * nv) : 0.0;
                if (cosines) cosines[((size_t)b * K + k) * (size_t)lv + j] = c[j];
            }
            qsort(c, (size_t)lv, sizeof(double), cmp_desc);
            const int n = top_n < lv ? top_n : lv;
            double sum = 0.0;
            for (int j = 0; j < n; ++j) sum += c[j];
            relevance[(size_t)b * K + k] = n > 0 ? sum / n : 0.0;
        }
        free(c);
        free(hd);
    }
}

/*
 * What a verify step hands back to the decoding loop.  The paper defines the
 * accepted length (Eq. 2) and is silent on the rest; this is the standard
 * speculative-decoding bookkeeping under the rule's decisions:
 *   - the first tau draft tokens are kept as they are (also at loosened or
 *     shift-tolerated positions: the later target rows were computed with
 *     exactly these tokens in the context);
 *   - if a position was rejected (tau < gamma) the target's own token at that
 *     position, y_tau, follows as the correction; with tau = gamma there is no
 *     further target row to take a bonus token from;
 *   - the cache keeps the accepted draft slots: new_kv_len = kv_len - gamma + tau
 *     (the correction token has no K/V yet; it is the next step's input).
 *
 *   draft, target   int32 [B, gamma]
 *   accept_len      int32 [B]
 *   kv_len          int32 [B] or NULL
 *   emitted         int32 [B, gamma]   tokens, -1 beyond n_emitted
 *   n_emitted       int32 [B]          min(tau + 1, gamma)
 *   new_kv_len      int32 [B]          (only with kv_len)
 */
void lvspec_oracle_emit(const int32_t *draft, const int32_t *target, const int32_t *accept_len,
                        const int32_t *kv_len, int B, int gamma, int32_t *emitted,
                        int32_t *n_emitted, int32_t *new_kv_len)
{
    for (int b = 0; b < B; ++b) {
        const int tau = accept_len[b];
        int n = 0;
        for (int i = 0; i < gamma; ++i) emitted[(size_t)b * gamma + i] = -1;
        for (int i = 0; i < tau; ++i) emitted[(size_t)b * gamma + n++] = draft[(size_t)b * gamma + i];
        if (tau < gamma) emitted[(size_t)b * gamma + n++] = target[(size_t)b * gamma + tau];
        n_emitted[b] = n;
        if (kv_len && new_kv_len) new_kv_len[b] = kv_len[b] - gamma + tau;
    }
}

/*
 * Draft-token trees: after every branch has been verified on its own (one
 * accepted length per branch), the branch with the longest accepted length is
 * kept; among equals the first.
 *   accept_len  int32 [B, R]  ->  best_branch int32 [B], best_len int32 [B]
 */
void lvspec_oracle_select_branch(const int32_t *accept_len, int B, int R, int32_t *best_branch,
                                 int32_t *best_len)
{
    for (int b = 0; b < B; ++b) {
        int best = 0;
        for (int r = 1; r < R; ++r)
            if (accept_len[(size_t)b * R + r] > accept_len[(size_t)b * R + best]) best = r;
        best_branch[b] = best;
        best_len[b] = accept_len[(size_t)b * R + best];
    }
}


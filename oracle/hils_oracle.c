/*
 * HiLS attention -- CPU oracle.  TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, double-precision restatement of the forward HiLS attention
 * operator, written from the paper's equations.  It shares no code with the
 * CUDA library and must never be linked, imported or called by it; only the
 * tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it computes, for a query at position i of sequence b (0-based positions
 * and chunk ids), for every KV group g and every query head h of that group:
 *
 *   Sec. 2.1      chunk of token j: c(j) = floor(j / S);
 *                 aligned left edge of the local window
 *                 l(i) = floor((i - W + 1) / S) * S  (floor toward -inf, clamped at 0);
 *                 candidate chunks C_i = {0, ..., l(i)/S - 1}.
 *   Eq. (surrogate top-k), App. C Eq. (HiLS GQA)
 *                 per-head surrogate score  s^h_c = scale * q^h . k'_c + b'_c,
 *                 group score u_c = max_h s^h_c, selected set I = the min(K, |C_i|)
 *                 candidates with the largest u_c (full stable sort; equal scores
 *                 go to the lower chunk id).
 *   Eq. (chunk mass)  local branch: logits scale * q^h . k_j for j in [l(i), i],
 *                 their log-sum-exp lambda_loc = log Z_swa and softmax output o_loc.
 *   Eq. (HiLS weights), App. C
 *                 every selected chunk gets its own softmax over its S tokens
 *                 (output o_c); chunks and the local branch are mixed with
 *                 alpha = softmax({s^h_c : c in I} U {lambda_loc}), using the
 *                 PER-HEAD surrogate score of each selected chunk:
 *                   out = alpha_loc * o_loc + sum_c alpha_c * o_c
 *                   lse = log( sum_c exp(s^h_c) + Z_swa ).
 *
 * No blocking, fusion or reordering beyond the steps above.  Inputs are fp32
 * or raw bf16 arrays, widened exactly to fp64 element by element; all
 * arithmetic is fp64 with libm exp/log.
 *
 * hils_oracle_landmarks (bottom of the file) is the step upstream of the operator: the
 * chunk summary of Proposition 3.1 (Eq. prop_q_c), pinned by tests/test_landmark_pins.py.
 *
 * Pinned by tests/test_oracle_pins.py (closed forms, invariants, library
 * attention on reductions, an independent dense-weight brute force).  The paper
 * prints no worked numeric example, so absolute values against the authors'
 * own implementation are unpinned; the semantics are pinned by those identities.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

typedef struct {
    int B, Hq, Hkv, Hl;   /* Hl in {Hkv, Hq}: number of landmark heads                */
    int Lq;               /* query rows stored per (b, head) in q                       */
    int T;                /* key/value tokens stored per (b, kv head)                   */
    int C;                /* landmark rows stored per (b, landmark head)                */
    int d, S, K, W;
    double scale;         /* <= 0 means 1/sqrt(d)                                       */
    int group_mode;       /* 0: u_c = max_h s^h_c (App. C); 1: max_h of softmax_c(s^h)  */
    int in_bf16;          /* 0: q,k,v,landmarks are float32; 1: raw bfloat16 (uint16)   */
} hils_oracle_params;

static long floordiv(long a, long b) {
    long q = a / b;
    if ((a % b != 0) && ((a < 0) != (b < 0))) q -= 1;
    return q;
}

/* element i of a float32 or raw-bfloat16 array, widened exactly to double */
static double ld(const void *base, size_t i, int bf16) {
    if (!bf16) return (double)((const float *)base)[i];
    uint32_t bits = (uint32_t)((const uint16_t *)base)[i] << 16;
    float f;
    memcpy(&f, &bits, sizeof f);
    return (double)f;
}

static double dotx(const void *a, size_t ia, const void *b, size_t ib, int n, int bf16) {
    double acc = 0.0;
    for (int t = 0; t < n; ++t) acc += ld(a, ia + t, bf16) * ld(b, ib + t, bf16);
    return acc;
}

typedef struct { double u; int c; } cand_t;

/* order: larger score first; equal scores -> lower chunk id first */
static int cand_cmp(const void *pa, const void *pb) {
    const cand_t *a = (const cand_t *)pa, *b = (const cand_t *)pb;
    if (a->u > b->u) return -1;
    if (a->u < b->u) return 1;
    return (a->c > b->c) - (a->c < b->c);
}

static int int_cmp(const void *pa, const void *pb) {
    int a = *(const int *)pa, b = *(const int *)pb;
    return (a > b) - (a < b);
}

/* softmax attention of one query over rows [lo, hi) of K/V; returns m + log Z, writes o[d] */
static double attend_span(const void *q, size_t iq, const void *k, const void *v, size_t ikv,
                          long lo, long hi, int d, double scale, int bf16, double *o, double *logits) {
    long n = hi - lo;
    double m = -INFINITY;
    for (long j = 0; j < n; ++j) {
        logits[j] = scale * dotx(q, iq, k, ikv + (size_t)(lo + j) * d, d, bf16);
        if (logits[j] > m) m = logits[j];
    }
    double Z = 0.0;
    for (int t = 0; t < d; ++t) o[t] = 0.0;
    for (long j = 0; j < n; ++j) {
        double p = exp(logits[j] - m);
        Z += p;
        for (int t = 0; t < d; ++t) o[t] += p * ld(v, ikv + (size_t)(lo + j) * d + t, bf16);
    }
    for (int t = 0; t < d; ++t) o[t] /= Z;
    return m + log(Z);
}

/*
 * Rows: row r is the query of sequence row_b[r], stored at q[row_b, :, row_qi[r], :],
 * sitting at sequence position row_pos[r].
 *
 * sel_mode 0: compute the selection (Eq. surrogate top-k) and write it to sel_idx/margin.
 * sel_mode 1: take sel_idx as given (ascending ids, -1 padded) and only attend.
 * do_attend 0: selection only (out/lse untouched).
 *
 * Outputs (any may be NULL): sel_idx [n_rows, Hkv, K] int32 ascending, -1 padded;
 * margin [n_rows, Hkv] = (K-th best group score) - ((K+1)-th best), +inf if none is cut;
 * out [n_rows, Hq, d]; lse [n_rows, Hq]; alpha [n_rows, Hq, K+1] (selected slots, then local).
 * Returns 0, or -1 on bad arguments.
 */
/* q_route: the routing query q-hat of Eq. (Q-Cal) (q-hat = q + W_up W_down h, computed upstream), same shape as q;
 * it replaces q in the surrogate scores s^h_c only (selection and fusion weights), never in the token-level
 * attention.  NULL means q-hat = q. */
static int rows_impl(const hils_oracle_params *p,
                     const void *q, const void *q_route, const void *k, const void *v,
                     const void *landmarks, const float *bias,
                     int64_t n_rows, const int32_t *row_b, const int32_t *row_qi,
                     const int64_t *row_pos,
                     int sel_mode, int do_attend,
                     int32_t *sel_idx, double *margin,
                     double *out, double *lse, double *alpha)
{
    const void *qs = q_route ? q_route : q;
    if (!p || p->Hq % p->Hkv != 0 || (p->Hl != p->Hkv && p->Hl != p->Hq) || p->S <= 0 ||
        p->K < 0 || p->W < 1 || !sel_idx)
        return -1;
    const int G = p->Hq / p->Hkv, d = p->d, S = p->S, K = p->K, bf = p->in_bf16;
    const double scale = p->scale > 0 ? p->scale : 1.0 / sqrt((double)d);
    const int64_t work = n_rows * p->Hkv;
    int status = 0;

#pragma omp parallel for schedule(dynamic, 4)
    for (int64_t w = 0; w < work; ++w) {
        const int64_t r = w / p->Hkv;
        const int g = (int)(w % p->Hkv);
        const int b = row_b[r];
        const long i = (long)row_pos[r];
        long lo = floordiv(i - p->W + 1, S) * S;             /* l(i), Sec. 2.1 */
        if (lo < 0) lo = 0;
        const int ncand = (int)(lo / S);                     /* |C_i| */
        if (i >= p->T || ncand > p->C) { status = -1; continue; }

        double *shat = (double *)malloc(sizeof(double) * (size_t)(G * (ncand > 0 ? ncand : 1)));
        cand_t *cand = (cand_t *)malloc(sizeof(cand_t) * (size_t)(ncand > 0 ? ncand : 1));
        double *logits = (double *)malloc(sizeof(double) * (size_t)((i - lo + 1) > S ? (i - lo + 1) : S));
        double *o_part = (double *)malloc(sizeof(double) * (size_t)d);
        double *lam = (double *)malloc(sizeof(double) * (size_t)(K + 1));
        double *o_all = (double *)malloc(sizeof(double) * (size_t)(K + 1) * (size_t)d);

        /* per-head surrogate scores s^h_c for every candidate chunk */
        for (int rr = 0; rr < G; ++rr) {
            const int h = g * G + rr;
            const int hl = (p->Hl == p->Hq) ? h : g;
            const size_t iq = (((size_t)b * p->Hq + h) * p->Lq + row_qi[r]) * d;
            for (int c = 0; c < ncand; ++c) {
                const size_t ilm = (((size_t)b * p->Hl + hl) * p->C + c) * d;
                double s = scale * dotx(qs, iq, landmarks, ilm, d, bf);
                if (bias) s += (double)bias[((size_t)b * p->Hl + hl) * p->C + c];
                shat[rr * ncand + c] = s;
            }
        }

        int32_t *sel = sel_idx + ((size_t)r * p->Hkv + g) * K;
        int n = 0;
        if (sel_mode == 0) {
            /* group score: max over the heads of the group (App. C) */
            for (int c = 0; c < ncand; ++c) { cand[c].c = c; cand[c].u = -INFINITY; }
            if (p->group_mode == 0) {
                for (int rr = 0; rr < G; ++rr)
                    for (int c = 0; c < ncand; ++c)
                        if (shat[rr * ncand + c] > cand[c].u) cand[c].u = shat[rr * ncand + c];
            } else {
                /* variant of Sec. 4.1: normalise each head's scores over the candidates first */
                for (int rr = 0; rr < G; ++rr) {
                    double m = -INFINITY, Z = 0.0;
                    for (int c = 0; c < ncand; ++c) if (shat[rr * ncand + c] > m) m = shat[rr * ncand + c];
                    for (int c = 0; c < ncand; ++c) Z += exp(shat[rr * ncand + c] - m);
                    for (int c = 0; c < ncand; ++c) {
                        double wgt = exp(shat[rr * ncand + c] - m) / Z;
                        if (wgt > cand[c].u) cand[c].u = wgt;
                    }
                }
            }
            qsort(cand, (size_t)ncand, sizeof(cand_t), cand_cmp);
            n = ncand < K ? ncand : K;
            if (margin)
                margin[(size_t)r * p->Hkv + g] = (ncand > K && K > 0) ? cand[K - 1].u - cand[K].u : INFINITY;
            for (int t = 0; t < n; ++t) sel[t] = cand[t].c;
            qsort(sel, (size_t)n, sizeof(int32_t), int_cmp);
            for (int t = n; t < K; ++t) sel[t] = -1;
        } else {
            for (int t = 0; t < K; ++t) if (sel[t] >= 0) n = t + 1;
        }

        if (do_attend) {
            const size_t ikv = ((size_t)b * p->Hkv + g) * (size_t)p->T * d;
            for (int rr = 0; rr < G; ++rr) {
                const int h = g * G + rr;
                const size_t iq = (((size_t)b * p->Hq + h) * p->Lq + row_qi[r]) * d;
                int nslot = 0;
                /* each selected chunk: its own softmax; mass comes from the surrogate score */
                for (int t = 0; t < n; ++t) {
                    const int c = sel[t];
                    if (c < 0) continue;
                    if (c >= ncand) { status = -1; continue; }
                    attend_span(q, iq, k, v, ikv, (long)c * S, (long)(c + 1) * S, d, scale, bf,
                                o_all + (size_t)nslot * d, logits);
                    lam[nslot] = shat[rr * ncand + c];
                    ++nslot;
                }
                /* local branch: tokens l(i)..i, mass is its own Z_swa */
                const double lam_loc = attend_span(q, iq, k, v, ikv, lo, i + 1, d, scale, bf, o_part, logits);
                double Mx = lam_loc;
                for (int t = 0; t < nslot; ++t) if (lam[t] > Mx) Mx = lam[t];
                double D = exp(lam_loc - Mx);
                for (int t = 0; t < nslot; ++t) D += exp(lam[t] - Mx);
                const double a_loc = exp(lam_loc - Mx) / D;
                if (out) {
                    double *orow = out + ((size_t)r * p->Hq + h) * d;
                    for (int x = 0; x < d; ++x) orow[x] = a_loc * o_part[x];
                    for (int t = 0; t < nslot; ++t) {
                        const double a = exp(lam[t] - Mx) / D;
                        for (int x = 0; x < d; ++x) orow[x] += a * o_all[(size_t)t * d + x];
                    }
                }
                if (lse) lse[(size_t)r * p->Hq + h] = Mx + log(D);
                if (alpha) {
                    double *ar = alpha + ((size_t)r * p->Hq + h) * (K + 1);
                    for (int t = 0; t < K; ++t) ar[t] = 0.0;
                    int slot = 0;
                    for (int t = 0; t < n; ++t) {
                        if (sel[t] < 0) continue;
                        ar[t] = exp(lam[slot] - Mx) / D;
                        ++slot;
                    }
                    ar[K] = a_loc;
                }
            }
        }
        free(shat); free(cand); free(logits); free(o_part); free(lam); free(o_all);
    }
    return status;
}

int hils_oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}


int hils_oracle_rows(const hils_oracle_params *p,
                     const void *q, const void *k, const void *v,
                     const void *landmarks, const float *bias,
                     int64_t n_rows, const int32_t *row_b, const int32_t *row_qi,
                     const int64_t *row_pos,
                     int sel_mode, int do_attend,
                     int32_t *sel_idx, double *margin,
                     double *out, double *lse, double *alpha)
{
    return rows_impl(p, q, NULL, k, v, landmarks, bias, n_rows, row_b, row_qi, row_pos, sel_mode, do_attend, sel_idx,
                     margin, out, lse, alpha);
}

int hils_oracle_rows_routed(const hils_oracle_params *p,
                            const void *q, const void *q_route, const void *k, const void *v,
                            const void *landmarks, const float *bias,
                            int64_t n_rows, const int32_t *row_b, const int32_t *row_qi,
                            const int64_t *row_pos,
                            int sel_mode, int do_attend,
                            int32_t *sel_idx, double *margin,
                            double *out, double *lse, double *alpha)
{
    return rows_impl(p, q, q_route, k, v, landmarks, bias, n_rows, row_b, row_qi, row_pos, sel_mode, do_attend,
                     sel_idx, margin, out, lse, alpha);
}

/*
 * Chunk summaries of Proposition 3.1 (Eq. LogSumExp linearization / Eq. prop_q_c).
 * For sequence b, landmark head hl (its KV head is hl / (Hl / Hkv)) and chunk c, with the chunk's
 * keys k_j, j in [c*S, min((c+1)*S, len_b)) and its learnable query q'_c = lq[b, hl, c, :]:
 *     s_j = scale * q'_c . k_j,   p = softmax_j(s),
 *     k'_c = sum_j p_j k_j                      (Attn(q'_c, K_c, K_c)),
 *     b'_c = - sum_j p_j log p_j                (entropy of p).
 * A chunk without tokens gets k' = 0, b' = 0.  The paper defines the summary for complete chunks; a
 * partial last chunk uses the tokens it has (reading: the softmax runs over the tokens present).
 *
 * lq [B,Hl,C,d] and k [B,Hkv,T,d] are fp32 or raw bf16 (in_bf16); seq_lens [B] or NULL (= T);
 * out_landmarks [B,Hl,C,d] and out_bias [B,Hl,C] are doubles.  Returns 0, or -1 for bad arguments.
 */
int hils_oracle_landmarks(const hils_oracle_params *p, const void *lq, const void *k, const int32_t *seq_lens,
                          double *out_landmarks, double *out_bias) {
    if (!p || !lq || !k || !out_landmarks || !out_bias) return -1;
    if (p->B < 1 || p->Hkv < 1 || p->Hl < 1 || p->Hl % p->Hkv != 0 || p->d < 1 || p->S < 1 || p->C < 0 || p->T < 0)
        return -1;
    const int per = p->Hl / p->Hkv;
    const double scale = p->scale > 0 ? p->scale : 1.0 / sqrt((double)p->d);
    const long total = (long)p->B * p->Hl * p->C;
#ifdef _OPENMP
#pragma omp parallel for schedule(static)
#endif
    for (long x = 0; x < total; ++x) {
        const int c = (int)(x % p->C);
        const int hl = (int)((x / p->C) % p->Hl);
        const int b = (int)(x / ((long)p->C * p->Hl));
        const int hkv = hl / per;
        long len = seq_lens ? seq_lens[b] : p->T;
        if (len > p->T) len = p->T;
        const long j0 = (long)c * p->S;
        long j1 = j0 + p->S;
        if (j1 > len) j1 = len;
        double *kp = out_landmarks + (size_t)x * p->d;
        for (int e = 0; e < p->d; ++e) kp[e] = 0.0;
        out_bias[x] = 0.0;
        if (j1 <= j0) continue;
        const size_t qoff = (size_t)x * p->d;
        const size_t koff = ((size_t)b * p->Hkv + hkv) * (size_t)p->T * p->d;
        const int n = (int)(j1 - j0);
        double *s = (double *)malloc(sizeof(double) * (size_t)n);
        double m = -INFINITY;
        for (int j = 0; j < n; ++j) {
            double acc = 0.0;
            for (int e = 0; e < p->d; ++e)
                acc += ld(lq, qoff + e, p->in_bf16) * ld(k, koff + (size_t)(j0 + j) * p->d + e, p->in_bf16);
            s[j] = scale * acc;
            if (s[j] > m) m = s[j];
        }
        double z = 0.0;
        for (int j = 0; j < n; ++j) z += exp(s[j] - m);
        double ent = 0.0;
        for (int j = 0; j < n; ++j) {
            const double pj = exp(s[j] - m) / z;
            if (pj > 0.0) ent -= pj * log(pj);
            for (int e = 0; e < p->d; ++e) kp[e] += pj * ld(k, koff + (size_t)(j0 + j) * p->d + e, p->in_bf16);
        }
        out_bias[x] = ent;
        free(s);
    }
    return 0;
}

/*
 * Backward of the operator: the gradient of a scalar loss through `out`, given dout = dLoss/dout.
 *
 * The paper states that the retrieval scores sit inside the forward attention weights so that the language-model
 * loss trains the landmarks (Sec. 3.2, below Eq. HiLS weights), but prints no backward equations: what follows is
 * the chain rule applied, step by step, to the forward above, with the selected set I held fixed (top-K has no
 * derivative) and q-hat = q.  For one query head (position i, head h), with slots t = selected chunks and the
 * local span, p_tj the softmax inside slot t, o_t = sum_j p_tj v_j, lambda_t the slot's log mass
 * (s^h_c = scale q.k'_c + b'_c for a selected chunk, log Z_swa = log sum_j exp(s_j) for the local span),
 * alpha = softmax_t(lambda), out = sum_t alpha_t o_t:
 *
 *   d alpha_t   = dout . o_t
 *   d lambda_t  = alpha_t (d alpha_t - sum_u alpha_u d alpha_u)            (softmax over the slots)
 *   d o_t       = alpha_t dout
 *   d v_j      += p_tj d o_t                                               (o_t = sum_j p_tj v_j)
 *   d p_tj      = d o_t . v_j
 *   d s_tj      = p_tj (d p_tj - sum_l p_tl d p_tl)                        (softmax inside the slot)
 *   local span only:  d s_tj += d lambda_t p_tj                            (lambda_loc = logsumexp_j s_j)
 *   selected chunk c: d q += scale d lambda_t k'_c,  d k'_c += scale d lambda_t q,  d b'_c += d lambda_t
 *   d q += scale sum_j d s_tj k_j,   d k_j += scale d s_tj q               (s_tj = scale q . k_j)
 *
 * Pinned by tests/test_backward_pins.py: central finite differences of the forward oracle in every input,
 * library autograd on the rows that reduce to causal softmax attention, and the K = 1 two-branch mix.
 *
 * Layouts: q, dout, dq [B, Hq, Lq, d]; k, v, dk, dv [B, Hkv, T, d]; landmarks, dlm [B, Hl, C, d];
 * bias, dbias [B, Hl, C]; sel_idx [B, Hkv, Lq, K] (ascending, -1 padded, as the forward wrote it).
 * Query row r sits at position pos0 + r.  The five gradient arrays are overwritten.  Returns 0 or -1.
 */
int hils_oracle_backward(const hils_oracle_params *p, const void *q, const void *k, const void *v,
                         const void *landmarks, const float *bias, const int32_t *sel_idx, int64_t pos0,
                         const double *dout, double *dq, double *dk, double *dv, double *dlm, double *dbias)
{
    if (!p || p->Hq % p->Hkv != 0 || (p->Hl != p->Hkv && p->Hl != p->Hq) || p->S <= 0 || p->K < 0 ||
        p->W < 1 || !sel_idx || !dout || !dq || !dk || !dv || !dlm || !dbias || pos0 < 0)
        return -1;
    const int G = p->Hq / p->Hkv, d = p->d, S = p->S, K = p->K, bf = p->in_bf16;
    const double scale = p->scale > 0 ? p->scale : 1.0 / sqrt((double)d);
    memset(dq, 0, sizeof(double) * (size_t)p->B * p->Hq * p->Lq * d);
    memset(dk, 0, sizeof(double) * (size_t)p->B * p->Hkv * p->T * d);
    memset(dv, 0, sizeof(double) * (size_t)p->B * p->Hkv * p->T * d);
    memset(dlm, 0, sizeof(double) * (size_t)p->B * p->Hl * p->C * d);
    memset(dbias, 0, sizeof(double) * (size_t)p->B * p->Hl * p->C);
    int status = 0;

    /* one (sequence, KV group) per thread: its slices of dk, dv, dlm, dbias belong to it alone */
#pragma omp parallel for schedule(dynamic, 1)
    for (int pair = 0; pair < p->B * p->Hkv; ++pair) {
        const int b = pair / p->Hkv, g = pair % p->Hkv;
        const size_t ikv = ((size_t)b * p->Hkv + g) * (size_t)p->T * d;
        const size_t max_span = (size_t)S * ((size_t)(p->W + S - 1) / S + 1);
        double *pr = (double *)malloc(sizeof(double) * (size_t)(K + 1) * max_span);   /* p_tj          */
        double *o = (double *)malloc(sizeof(double) * (size_t)(K + 1) * d);           /* o_t           */
        double *lam = (double *)malloc(sizeof(double) * (size_t)(K + 1));
        double *alpha = (double *)malloc(sizeof(double) * (size_t)(K + 1));
        double *dalpha = (double *)malloc(sizeof(double) * (size_t)(K + 1));
        double *dp = (double *)malloc(sizeof(double) * max_span);
        long *lo_t = (long *)malloc(sizeof(long) * (size_t)(K + 1));
        long *n_t = (long *)malloc(sizeof(long) * (size_t)(K + 1));
        int *chunk_t = (int *)malloc(sizeof(int) * (size_t)(K + 1));

        for (int r = 0; r < p->Lq; ++r) {
            const long i = (long)(pos0 + r);
            long lo = floordiv(i - p->W + 1, S) * S;
            if (lo < 0) lo = 0;
            const int ncand = (int)(lo / S);
            if (i >= p->T || ncand > p->C) { status = -1; continue; }
            const int32_t *sel = sel_idx + (((size_t)b * p->Hkv + g) * p->Lq + r) * K;

            for (int rr = 0; rr < G; ++rr) {
                const int h = g * G + rr;
                const int hl = (p->Hl == p->Hq) ? h : g;
                const size_t iq = (((size_t)b * p->Hq + h) * p->Lq + r) * d;
                const double *dor = dout + iq;

                /* ---- forward, keeping what the derivative needs */
                int nslot = 0;
                for (int t = 0; t < K; ++t) {
                    const int c = sel[t];
                    if (c < 0) continue;
                    if (c >= ncand) { status = -1; continue; }
                    chunk_t[nslot] = c; lo_t[nslot] = (long)c * S; n_t[nslot] = S;
                    const size_t ilm = (((size_t)b * p->Hl + hl) * p->C + c) * d;
                    lam[nslot] = scale * dotx(q, iq, landmarks, ilm, d, bf);
                    if (bias) lam[nslot] += (double)bias[((size_t)b * p->Hl + hl) * p->C + c];
                    ++nslot;
                }
                chunk_t[nslot] = -1; lo_t[nslot] = lo; n_t[nslot] = i + 1 - lo;        /* the local span */
                ++nslot;
                for (int t = 0; t < nslot; ++t) {
                    double *pt = pr + (size_t)t * max_span, *ot = o + (size_t)t * d;
                    double m = -INFINITY, Z = 0.0;
                    for (long j = 0; j < n_t[t]; ++j) {
                        pt[j] = scale * dotx(q, iq, k, ikv + (size_t)(lo_t[t] + j) * d, d, bf);
                        if (pt[j] > m) m = pt[j];
                    }
                    for (long j = 0; j < n_t[t]; ++j) { pt[j] = exp(pt[j] - m); Z += pt[j]; }
                    for (int x = 0; x < d; ++x) ot[x] = 0.0;
                    for (long j = 0; j < n_t[t]; ++j) {
                        pt[j] /= Z;
                        for (int x = 0; x < d; ++x) ot[x] += pt[j] * ld(v, ikv + (size_t)(lo_t[t] + j) * d + x, bf);
                    }
                    if (chunk_t[t] < 0) lam[t] = m + log(Z);
                }
                double Mx = -INFINITY, Dn = 0.0;
                for (int t = 0; t < nslot; ++t) if (lam[t] > Mx) Mx = lam[t];
                for (int t = 0; t < nslot; ++t) Dn += exp(lam[t] - Mx);
                for (int t = 0; t < nslot; ++t) alpha[t] = exp(lam[t] - Mx) / Dn;

                /* ---- backward */
                double mix = 0.0;                                   /* sum_u alpha_u d alpha_u */
                for (int t = 0; t < nslot; ++t) {
                    dalpha[t] = 0.0;
                    for (int x = 0; x < d; ++x) dalpha[t] += dor[x] * o[(size_t)t * d + x];
                    mix += alpha[t] * dalpha[t];
                }
                double *dqr = dq + iq;
                for (int t = 0; t < nslot; ++t) {
                    const double *pt = pr + (size_t)t * max_span;
                    const double dlam = alpha[t] * (dalpha[t] - mix);
                    double inner = 0.0;                             /* sum_l p_tl d p_tl */
                    for (long j = 0; j < n_t[t]; ++j) {
                        dp[j] = 0.0;
                        for (int x = 0; x < d; ++x)
                            dp[j] += alpha[t] * dor[x] * ld(v, ikv + (size_t)(lo_t[t] + j) * d + x, bf);
                        inner += pt[j] * dp[j];
                    }
                    for (long j = 0; j < n_t[t]; ++j) {
                        const size_t row = ikv + (size_t)(lo_t[t] + j) * d;
                        double ds = pt[j] * (dp[j] - inner);
                        if (chunk_t[t] < 0) ds += dlam * pt[j];
                        for (int x = 0; x < d; ++x) {
                            dv[row + x] += pt[j] * alpha[t] * dor[x];
                            dqr[x] += scale * ds * ld(k, row + x, bf);
                            dk[row + x] += scale * ds * ld(q, iq + x, bf);
                        }
                    }
                    if (chunk_t[t] >= 0) {
                        const size_t ilm = (((size_t)b * p->Hl + hl) * p->C + chunk_t[t]) * d;
                        for (int x = 0; x < d; ++x) {
                            dqr[x] += scale * dlam * ld(landmarks, ilm + x, bf);
                            dlm[ilm + x] += scale * dlam * ld(q, iq + x, bf);
                        }
                        dbias[((size_t)b * p->Hl + hl) * p->C + chunk_t[t]] += dlam;
                    }
                }
            }
        }
        free(pr); free(o); free(lam); free(alpha); free(dalpha); free(dp); free(lo_t); free(n_t); free(chunk_t);
    }
    return status;
}

/*
 * rr_oracle.c -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, sequential-in-spirit CPU statement of what one rectified
 * Mixture-of-Experts layer computes (arXiv 2402.12399, "Rectify-Router"):
 * top-k routing with a per-expert capacity, Intra-GPU Rectification (IR),
 * Fill-in Rectification (FR), the combine weights, the SwiGLU expert FFN
 * forward and its backward, the gate projection that produces the logits,
 * and the router's load-balance loss.  All floating point is fp64 on the exact
 * fp32 / bf16 input values; every comparison that decides an integer is
 * made on the raw fp32 logits (with the softmax-valued FR key: on a single-
 * precision softmax whose every operation is fixed, see rro_softmax32).
 *
 * It shares no code with the CUDA library and must never be linked, loaded
 * or called by it.  Only the tests, the smoke check and the benchmark's CPU
 * baseline leg may use it.
 *
 * Each function cites the passage of the paper it follows.  Where the paper
 * is silent the chosen reading is stated at the function.
 *
 * OpenMP is used only over independent tokens / rows so that the timed CPU
 * baseline may use the host cores; results do not depend on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define RRO_IR 1u
#define RRO_FR 2u
#define RRO_SCORE 4u /* overflow drops the lowest scores instead of the latest tokens */
#define RRO_LOCALCAP 16u /* capacity applies per (source group, expert): C/G slots each, instead of C over all tokens */
#define RRO_FRSOFT 8u /* FR ranks an expert's nominees by softmax value g_ie instead of raw logit a_ie */

#define RRO_OK 0
#define RRO_INVALID 1
#define RRO_NONFINITE 2
#define RRO_NOMEM 3

/* element type of hidden / weights / dout handed to the layer functions */
#define RRO_F32 0
#define RRO_BF16 1

int rro_num_threads(void)
{
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

void rro_set_num_threads(int n)
{
#ifdef _OPENMP
    if (n > 0) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* The order used everywhere a "highest score" is asked for: larger raw logit
 * first, and on equal logits (float equality, so -0 == +0) the lower index.
 * Section 3, Eq. 1 fixes "top-k scores"; the tie rule is this build's. */
static int precedes(float a, int ia, float b, int ib)
{
    if (a > b) return 1;
    if (a < b) return 0;
    return ia < ib;
}

/*
 * The softmax value g_ie = e^{a_ie} / sum_j e^{a_ij} in single precision with
 * every operation and its order fixed, so that any IEEE-754 machine obtains the
 * same 32 bits.  Appendix A calls g_ij the "routing scores"; read that way, the
 * second stage of FR (Section 4.2) compares g values of DIFFERENT tokens, and a
 * comparison that decides an integer has to be reproducible, which an
 * unspecified library exp is not.  The recipe (all operations round to nearest
 * even, no contraction other than the fused multiply-adds written out):
 *   m   = max_j a_ij
 *   t_j = max(a_ij - m, -80)                        (keeps every result normal)
 *   n   = rint(t_j * log2(e)),  r = fma(-n, ln2_hi, t_j),  r = fma(-n, ln2_lo, r)
 *   p   = Taylor polynomial of e^r, degree 7, Horner form with fma,
 *         coefficients 1/q! rounded to single precision   (|r| <= 0.35: error < 1e-8)
 *   e_j = p * 2^n                                   (exact scaling)
 *   Z   = (((e_0 + e_1) + e_2) + ...) + e_{E-1}     (index order)
 *   g_ie = e_e / Z
 * ln2_hi = 0x1.62e4p-1 has few enough digits for n * ln2_hi to be exact; ln2_lo =
 * 0x1.7f7d1cp-20 is the rest of ln 2 (the classical two-constant range reduction).
 */
static float exp32_fixed(float t)
{
    if (t < -80.0f) t = -80.0f;
    const float n = rintf(t * 0x1.715476p+0f);
    float r = fmaf(-n, 0x1.62e4p-1f, t);
    r = fmaf(-n, 0x1.7f7d1cp-20f, r);
    float p = 0x1.a01a02p-13f;      /* 1/7! */
    p = fmaf(p, r, 0x1.6c16c2p-10f); /* 1/6! */
    p = fmaf(p, r, 0x1.111112p-7f);  /* 1/5! */
    p = fmaf(p, r, 0x1.555556p-5f);  /* 1/4! */
    p = fmaf(p, r, 0x1.555556p-3f);  /* 1/3! */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    return ldexpf(p, (int)n);
}

/* g[0..E-1] = the fixed single-precision softmax of one row of logits (see above). */
void rro_softmax32(const float *a, int E, float *g)
{
    float m = a[0];
    for (int j = 1; j < E; ++j)
        if (a[j] > m) m = a[j];
    float Z = 0.0f;
    for (int j = 0; j < E; ++j) {
        g[j] = exp32_fixed(a[j] - m);
        Z = (j == 0) ? g[0] : Z + g[j];
    }
    for (int j = 0; j < E; ++j) g[j] = g[j] / Z;
}

/* Argument rules shared by the routing entry points. */
static int check_shape(int T, int E, int k, int C, int G, unsigned mode)
{
    if (T < 0 || E < 1 || k < 1 || C < 0 || G < 1) return RRO_INVALID;
    if (k > E) return RRO_INVALID;
    if ((mode & RRO_FR) && k >= E) return RRO_INVALID; /* FR needs a (k+1)-th expert */
    if (mode & ~(RRO_IR | RRO_FR | RRO_SCORE | RRO_FRSOFT | RRO_LOCALCAP)) return RRO_INVALID;
    if ((mode & RRO_LOCALCAP) && C % G != 0) return RRO_INVALID; /* every group owns C/G slots of each expert */
    if ((mode & RRO_FRSOFT) && !(mode & RRO_FR)) return RRO_INVALID; /* the key belongs to FR */
    if (T % G != 0 || E % G != 0) return RRO_INVALID;
    return RRO_OK;
}

/*
 * Combine weights of one token (Section 3 Eq. 2; Section 4.1 Eq. 3).
 *
 * The token's live routes are: its top-k routes that obtained a slot
 * (multiplicity 1), its fill-in route if it was placed (multiplicity 1;
 * Section 4.2 reads FR as a top-(k+1) router, so the fill route simply joins
 * Eq. 2's sum), and its IR route (multiplicity k-|R_i| = number of dropped
 * top-k routings, Eq. 3).  w_r = mu_r e^{a_r} / sum_r' mu_r' e^{a_r'};
 * the max logit of the token is subtracted first, which changes nothing
 * mathematically.  Columns: 0..k-1 top-k ranks, k fill-in, k+1 IR.
 */
static void token_weights(const float *a_i, int E, int k, const int32_t *topk_expert_i,
                          const int32_t *route_slot_i, int d_i, int h_i, double *w_i)
{
    double m = a_i[0];
    for (int j = 1; j < E; ++j)
        if ((double)a_i[j] > m) m = a_i[j];
    double num[64 + 2];
    double den = 0.0;
    for (int r = 0; r <= k; ++r) {
        num[r] = 0.0;
        if (route_slot_i[r] >= 0) {
            num[r] = exp((double)a_i[topk_expert_i[r]] - m);
            den += num[r];
        }
    }
    num[k + 1] = 0.0;
    if (h_i >= 0) {
        num[k + 1] = (double)d_i * exp((double)a_i[h_i] - m);
        den += num[k + 1];
    }
    for (int r = 0; r < k + 2; ++r) w_i[r] = (den > 0.0) ? num[r] / den : 0.0;
}

/*
 * rro_weights: recompute combine weights from logits for FIXED routing tables.
 * Used by the routing oracle itself and by gradient tests that perturb the
 * logits while the routing decisions stay frozen.
 */
int rro_weights(const float *logits, int T, int E, int k, const int32_t *topk_expert,
                const int32_t *route_slot, const int32_t *drop_count, const int32_t *ir_expert,
                double *combine_w)
{
    if (k > 64) return RRO_INVALID;
    for (int i = 0; i < T; ++i)
        token_weights(logits + (size_t)i * E, E, k, topk_expert + (size_t)i * (k + 1),
                      route_slot + (size_t)i * (k + 1), drop_count[i], ir_expert[i],
                      combine_w + (size_t)i * (k + 2));
    return RRO_OK;
}

/*
 * rro_route: the routing procedure.
 *
 *  logits        [T,E] fp32, a_ij of Eq. 1
 *  capacity C    slots per expert (Section 3, "capacity"), applied over all T tokens
 *  G             number of groups ("GPUs" of Section 4.1); token i is in group
 *                i / (T/G), group g owns experts [g E/G, (g+1) E/G)
 *  mode          bit 0 = IR, bit 1 = FR, bit 2 = score-priority dropping (the other reading of
 *                Section 3: a full expert drops the tokens with the lowest scores, not the latest),
 *                bit 3 = FR ranks nominees by softmax value (Appendix A's "routing scores")
 *                instead of raw logit; needs bit 1,
 *                bit 4 = per-source capacity: Section 3 places the experts on G devices and
 *                defines the capacity from "the number of tokens"; a device that routes its own
 *                batch sees only its T/G tokens, so each expert grants every source group C/G
 *                slots of its own (slots [g C/G, (g+1) C/G) belong to group g) and queues,
 *                drops, padding and fill-in are all counted per (group, expert).  Needs G | C.
 *
 * Outputs (caller-allocated):
 *  topk_expert   [T,k+1]  experts of token i ordered by (logit desc, index asc);
 *                         column k is the (k+1)-th expert (FR's nominee), -1 if E == k
 *  route_slot    [T,k+1]  slot obtained at that expert, -1 if none
 *  slot_token    [E,C]    token in that slot, -1 = padding
 *  slot_rank     [E,C]    rank r of the routing that filled it (k = fill-in), -1 = padding
 *  drop_count    [T]      d_i = number of the token's top-k routings that were dropped
 *  ir_expert     [T]      IR expert h_i, -1 if the token takes no IR route
 *  ir_pos        [T]      position in h_i's IR list, -1 if none
 *  ir_offset     [E+1]    exclusive prefix of IR list lengths
 *  ir_token      [T]      IR lists, expert after expert; entries past ir_offset[E] are -1
 *  expert_count  [E]      occupied slots of each expert (kept + filled); they are slots 0..count-1
 *                         (with per-source capacity: the total over the groups' segments, each
 *                         segment filled from its first slot)
 *  n_routed      [E]      n_e: top-k routings addressed to e before the capacity cut
 *  row_offset    [E+1]    live rows (occupied slots then IR list) of expert e are rows
 *                         row_offset[e] .. row_offset[e+1]-1 of the compact row space
 *  row_token     [E*C+T]  token of each live row, -1 past row_offset[E]
 *  row_weight    [E*C+T]  combine weight of each live row (fp64), 0 past the end
 *  token_rows    [T,k+2]  row of each of the token's routes (columns as combine_w), -1 if none
 *  combine_w     [T,k+2]  fp64 weights
 */
int rro_route(const float *logits, int T, int E, int k, int C, int G, unsigned mode,
              int32_t *topk_expert, int32_t *route_slot, int32_t *slot_token, int8_t *slot_rank,
              int32_t *drop_count, int32_t *ir_expert, int32_t *ir_pos, int32_t *ir_offset,
              int32_t *ir_token, int32_t *expert_count, int32_t *n_routed, int32_t *row_offset,
              int32_t *row_token, double *row_weight, int32_t *token_rows, double *combine_w)
{
    int rc = check_shape(T, E, k, C, G, mode);
    if (rc) return rc;
    if (k > 64) return RRO_INVALID;
    for (size_t n = 0; n < (size_t)T * E; ++n)
        if (!isfinite(logits[n])) return RRO_NONFINITE;

    const int K1 = k + 1;
    const int tokens_per_group = T / G;
    const int experts_per_group = E / G;
    /* Capacity segments: one over all tokens, or one per source group. Segment s of
     * every expert owns slots [s Cs, (s+1) Cs) and serves tokens [s Ts, (s+1) Ts). */
    const int S = (mode & RRO_LOCALCAP) ? G : 1;
    const int Cs = C / S;
    const int Ts = T / S;

    /* Eq. 1: R_i = argtopk_j a_ij, extended by one place for FR's nominee
     * (Section 4.2, first stage: each token picks its (k+1)-th ranked expert). */
    for (int i = 0; i < T; ++i) {
        const float *a = logits + (size_t)i * E;
        int32_t *sel = topk_expert + (size_t)i * K1;
        for (int r = 0; r < K1; ++r) {
            int best = -1;
            for (int j = 0; j < E; ++j) {
                int taken = 0;
                for (int q = 0; q < r; ++q)
                    if (sel[q] == j) taken = 1;
                if (taken) continue;
                if (best < 0 || precedes(a[j], j, a[best], best)) best = j;
            }
            sel[r] = best; /* -1 only when r == k == E */
        }
    }

    /* Section 3, "Dropped Tokens and Padding": every expert accepts at most C
     * tokens; what exceeds it is dropped, what is missing is padding.
     * Reading: first-routing choices of all tokens are served before any
     * second-routing choice (Section 4.1 speaks of a token's first and second
     * routing as separate events), and inside one routing tokens queue in token
     * order (Fig. 1 draws one queue per expert). */
    for (size_t n = 0; n < (size_t)E * C; ++n) { slot_token[n] = -1; slot_rank[n] = -1; }
    for (size_t n = 0; n < (size_t)T * K1; ++n) route_slot[n] = -1;
    for (int i = 0; i < T; ++i) drop_count[i] = 0;
    int32_t *count = (int32_t *)calloc((size_t)S * E, sizeof(int32_t)); /* queue length per (segment, expert) */
    int32_t *occ = (int32_t *)calloc((size_t)S * E, sizeof(int32_t));   /* occupied slots per (segment, expert) */
    if (!count || !occ) return RRO_NOMEM;
    for (int r = 0; r < k && !(mode & RRO_SCORE); ++r) {
        for (int i = 0; i < T; ++i) {
            int e = topk_expert[(size_t)i * K1 + r];
            int sg = (S == 1) ? 0 : i / Ts;
            int pos = count[sg * E + e]++;
            if (pos < Cs) {
                pos += sg * Cs;
                route_slot[(size_t)i * K1 + r] = pos;
                slot_token[(size_t)e * C + pos] = i;
                slot_rank[(size_t)e * C + pos] = (int8_t)r;
            } else {
                drop_count[i] += 1; /* |R_i| = k - d_i <= k */
            }
        }
    }
    /* The other reading of Section 3 ("drop tokens with the lowest routing
     * scores"): routings are still served rank after rank, but when the r-th
     * choices addressed to expert e exceed what is left of its capacity, the
     * ones with the highest scores a_ie stay (ties: lower token) and the rest
     * are dropped.  Those that stay take the next slots in ascending token
     * order, as the kept and the filled tokens do in the other reading. */
    if (mode & RRO_SCORE) {
        int32_t *cand = (int32_t *)malloc(((size_t)T + 1) * sizeof(int32_t));
        char *stays = (char *)malloc((size_t)T + 1);
        if (!cand || !stays) return RRO_NOMEM;
        for (int r = 0; r < k; ++r) {
            for (int se = 0; se < S * E; ++se) {
                int sg = se / E, e = se % E;
                int n = 0;
                for (int i = sg * Ts; i < (sg + 1) * Ts; ++i)
                    if (topk_expert[(size_t)i * K1 + r] == e) cand[n++] = i;
                int taken = count[se] < Cs ? count[se] : Cs; /* slots used by lower ranks */
                int left = Cs - taken;
                int take = n < left ? n : left;
                memset(stays, 0, (size_t)n + 1);
                for (int t = 0; t < take; ++t) { /* best remaining by (a_ie desc, i asc) */
                    int best = -1;
                    for (int q = 0; q < n; ++q) {
                        if (stays[q]) continue;
                        if (best < 0 || precedes(logits[(size_t)cand[q] * E + e], cand[q],
                                                 logits[(size_t)cand[best] * E + e], cand[best]))
                            best = q;
                    }
                    stays[best] = 1;
                }
                int pos = sg * Cs + taken;
                for (int q = 0; q < n; ++q) { /* cand[] is in ascending token order */
                    int i = cand[q];
                    if (stays[q]) {
                        route_slot[(size_t)i * K1 + r] = pos;
                        slot_token[(size_t)e * C + pos] = i;
                        slot_rank[(size_t)e * C + pos] = (int8_t)r;
                        ++pos;
                    } else {
                        drop_count[i] += 1;
                    }
                }
                count[se] += n;
            }
        }
        free(cand);
        free(stays);
    }
    for (int e = 0; e < E; ++e) {
        n_routed[e] = 0;
        expert_count[e] = 0;
        for (int sg = 0; sg < S; ++sg) {
            occ[sg * E + e] = count[sg * E + e] < Cs ? count[sg * E + e] : Cs; /* kept */
            n_routed[e] += count[sg * E + e];
            expert_count[e] += occ[sg * E + e];
        }
    }
    free(count);

    /* Section 4.1 (IR): a token with at least one dropped routing goes, once,
     * to the best-scoring expert of its own group; no capacity applies, and the
     * experts already in R_i are not excluded (with G = 1 this must be exactly
     * top-1 routing).  Lists are in token order. */
    for (int i = 0; i < T; ++i) { ir_expert[i] = -1; ir_pos[i] = -1; ir_token[i] = -1; }
    for (int e = 0; e <= E; ++e) ir_offset[e] = 0;
    if (mode & RRO_IR) {
        for (int i = 0; i < T; ++i) {
            if (drop_count[i] == 0) continue;
            const float *a = logits + (size_t)i * E;
            int g = i / tokens_per_group;
            int h = g * experts_per_group;
            for (int j = h + 1; j < (g + 1) * experts_per_group; ++j)
                if (precedes(a[j], j, a[h], h)) h = j;
            ir_expert[i] = h;
            ir_offset[h + 1] += 1;
        }
        for (int e = 0; e < E; ++e) ir_offset[e + 1] += ir_offset[e];
        int32_t *fill = (int32_t *)calloc((size_t)E, sizeof(int32_t));
        if (!fill) return RRO_NOMEM;
        for (int i = 0; i < T; ++i) {
            int h = ir_expert[i];
            if (h < 0) continue;
            ir_pos[i] = fill[h]++;
            ir_token[ir_offset[h] + ir_pos[i]] = i;
        }
        free(fill);
    }

    /* Section 4.2 (FR): stage one, every token nominates its (k+1)-th expert;
     * stage two, expert e has v_e = C - kept_e padding slots and gives them to
     * its nominees with the highest scores (ties: lower token).  The chosen
     * tokens occupy slots kept_e, kept_e+1, ... in ascending token order, which
     * makes FR coincide with a top-(k+1) router whenever nobody is refused. */
    if (mode & RRO_FR) {
        int32_t *nominee = (int32_t *)malloc(((size_t)T + 1) * sizeof(int32_t));
        char *chosen = (char *)malloc((size_t)T + 1);
        /* score[i] = what token i is ranked by at the expert it nominates: the raw
         * logit a_ie (Section 3 calls a_ij "the score"), or with RRO_FRSOFT the
         * softmax value g_ie (Appendix A's "routing scores"), in the fixed single
         * precision of rro_softmax32. */
        float *score = (float *)malloc(((size_t)T + 1) * sizeof(float));
        float *g_row = (float *)malloc((size_t)E * sizeof(float));
        if (!nominee || !chosen || !score || !g_row) return RRO_NOMEM;
        for (int i = 0; i < T; ++i) {
            int e = topk_expert[(size_t)i * K1 + k];
            if (mode & RRO_FRSOFT) {
                rro_softmax32(logits + (size_t)i * E, E, g_row);
                score[i] = g_row[e];
            } else {
                score[i] = logits[(size_t)i * E + e];
            }
        }
        for (int se = 0; se < S * E; ++se) {
            int sg = se / E, e = se % E;
            int n = 0;
            for (int i = sg * Ts; i < (sg + 1) * Ts; ++i)
                if (topk_expert[(size_t)i * K1 + k] == e) nominee[n++] = i;
            int v = Cs - occ[se];
            int take = n < v ? n : v;
            /* nominee[] is in ascending token order; pick `take` of them by
             * repeated selection of the best remaining (a_ie desc, i asc). */
            memset(chosen, 0, (size_t)n + 1);
            for (int t = 0; t < take; ++t) {
                int best = -1;
                for (int q = 0; q < n; ++q) {
                    if (chosen[q]) continue;
                    if (best < 0 || precedes(score[nominee[q]], nominee[q], score[nominee[best]], nominee[best]))
                        best = q;
                }
                chosen[best] = 1;
            }
            int s = sg * Cs + occ[se];
            for (int q = 0; q < n; ++q) {
                if (!chosen[q]) continue;
                int i = nominee[q];
                route_slot[(size_t)i * K1 + k] = s;
                slot_token[(size_t)e * C + s] = i;
                slot_rank[(size_t)e * C + s] = (int8_t)k;
                ++s;
            }
            expert_count[e] += s - (sg * Cs + occ[se]);
            occ[se] = s - sg * Cs;
        }
        free(nominee);
        free(chosen);
        free(score);
        free(g_row);
    }

    /* Eq. 2 / Eq. 3 weights. */
    rro_weights(logits, T, E, k, topk_expert, route_slot, drop_count, ir_expert, combine_w);

    /* Compact row space: the rows an expert actually computes. */
    row_offset[0] = 0;
    for (int e = 0; e < E; ++e)
        row_offset[e + 1] = row_offset[e] + expert_count[e] + (ir_offset[e + 1] - ir_offset[e]);
    size_t Rmax = (size_t)E * C + (size_t)T;
    for (size_t n = 0; n < Rmax; ++n) { row_token[n] = -1; row_weight[n] = 0.0; }
    for (size_t n = 0; n < (size_t)T * (k + 2); ++n) token_rows[n] = -1;
    for (int i = 0; i < T; ++i) {
        for (int r = 0; r <= k; ++r) {
            int s = route_slot[(size_t)i * K1 + r];
            if (s < 0) continue;
            int e = topk_expert[(size_t)i * K1 + r];
            int row = row_offset[e]; /* + the number of occupied slots of e below slot s */
            for (int sg = 0; sg < s / Cs; ++sg) row += occ[sg * E + e];
            row += s % Cs;
            token_rows[(size_t)i * (k + 2) + r] = row;
            row_token[row] = i;
            row_weight[row] = combine_w[(size_t)i * (k + 2) + r];
        }
        if (ir_expert[i] >= 0) {
            int h = ir_expert[i];
            int row = row_offset[h] + expert_count[h] + ir_pos[i];
            token_rows[(size_t)i * (k + 2) + k + 1] = row;
            row_token[row] = i;
            row_weight[row] = combine_w[(size_t)i * (k + 2) + k + 1];
        }
    }
    free(occ);
    return RRO_OK;
}

/* ---------------------------------------------------------------------- */
/* Expert FFN.  Section 5.1 ("Model"): each expert is a copy of the dense
 * model's FFN, a LLaMA-style gated MLP without biases:
 *     E_j(x) = W2_j ( silu(W1_j x) * (W3_j x) ),  silu(z) = z / (1 + e^-z).
 * Weight layout: W1,W3 [E][d_ff][d], W2 [E][d][d_ff], row-major.           */

static inline double ld(const void *p, size_t n, int dtype)
{
    if (dtype == RRO_BF16) {
        uint32_t bits = (uint32_t)((const uint16_t *)p)[n] << 16;
        float f;
        memcpy(&f, &bits, 4);
        return (double)f;
    }
    return (double)((const float *)p)[n];
}

static double silu(double z) { return z / (1.0 + exp(-z)); }
static double dsilu(double z)
{
    double s = 1.0 / (1.0 + exp(-z));
    return s * (1.0 + z * (1.0 - s));
}

/* h1 = W1_e x, h3 = W3_e x, act = silu(h1)*h3, y = W2_e act. */
static void expert_forward(const double *x, const void *W1, const void *W3, const void *W2, int e,
                           int d, int d_ff, int dtype, double *h1, double *h3, double *act,
                           double *y)
{
    size_t w13 = (size_t)e * d_ff * d, w2 = (size_t)e * d * d_ff;
    for (int f = 0; f < d_ff; ++f) {
        double s1 = 0.0, s3 = 0.0;
        for (int c = 0; c < d; ++c) {
            s1 += ld(W1, w13 + (size_t)f * d + c, dtype) * x[c];
            s3 += ld(W3, w13 + (size_t)f * d + c, dtype) * x[c];
        }
        h1[f] = s1;
        h3[f] = s3;
        act[f] = silu(s1) * s3;
    }
    for (int n = 0; n < d; ++n) {
        double s = 0.0;
        for (int f = 0; f < d_ff; ++f) s += ld(W2, w2 + (size_t)n * d_ff + f, dtype) * act[f];
        y[n] = s;
    }
}

/* routes of a token: expert and multiplicity per column of combine_w */
static int route_expert(int k, const int32_t *topk_expert_i, const int32_t *route_slot_i, int h_i,
                        int r)
{
    if (r <= k) return route_slot_i[r] >= 0 ? topk_expert_i[r] : -1;
    return h_i;
}

/*
 * rro_forward_tokens: out_i = sum_r w_r E_{e_r}(x_i) over the live routes of
 * token i (Eq. 2, Eq. 3), for the tokens listed in `tokens` (n_tok of them).
 * Tokens without a live route give 0 (Section 3: they reach the next layer
 * through the residual connection only, which is outside this layer).  Weights are recomputed from the logits, so
 * the tables may be held fixed while logits vary.
 *   out    [n_tok, d] fp64
 *   y_rows [n_tok, k+2, d] fp64 or NULL: the unweighted expert outputs E_{e_r}(x_i)
 */
int rro_forward_tokens(const void *hidden, const void *W1, const void *W3, const void *W2,
                       int dtype, const float *logits, int T, int E, int k, int d, int d_ff,
                       const int32_t *topk_expert, const int32_t *route_slot,
                       const int32_t *drop_count, const int32_t *ir_expert, const int32_t *tokens,
                       int n_tok, double *out, double *y_rows)
{
    if (k > 64) return RRO_INVALID;
    int failed = 0;
#pragma omp parallel
    {
        double *x = (double *)malloc(sizeof(double) * (size_t)d);
        double *y = (double *)malloc(sizeof(double) * (size_t)d);
        double *h1 = (double *)malloc(sizeof(double) * (size_t)d_ff * 3);
        if (!x || !y || !h1) {
#pragma omp atomic write
            failed = 1;
        } else {
            double *h3 = h1 + d_ff, *act = h3 + d_ff;
#pragma omp for schedule(dynamic, 1)
            for (int t = 0; t < n_tok; ++t) {
                int i = tokens[t];
                double w[64 + 2];
                token_weights(logits + (size_t)i * E, E, k, topk_expert + (size_t)i * (k + 1),
                              route_slot + (size_t)i * (k + 1), drop_count[i], ir_expert[i], w);
                for (int c = 0; c < d; ++c) x[c] = ld(hidden, (size_t)i * d + c, dtype);
                double *o = out + (size_t)t * d;
                for (int c = 0; c < d; ++c) o[c] = 0.0;
                for (int r = 0; r < k + 2; ++r) {
                    int e = route_expert(k, topk_expert + (size_t)i * (k + 1),
                                         route_slot + (size_t)i * (k + 1), ir_expert[i], r);
                    double *yr = y_rows ? y_rows + ((size_t)t * (k + 2) + r) * d : NULL;
                    if (e < 0) {
                        if (yr) for (int c = 0; c < d; ++c) yr[c] = 0.0;
                        continue;
                    }
                    expert_forward(x, W1, W3, W2, e, d, d_ff, dtype, h1, h3, act, y);
                    for (int c = 0; c < d; ++c) o[c] += w[r] * y[c];
                    if (yr) for (int c = 0; c < d; ++c) yr[c] = y[c];
                }
            }
        }
        free(x); free(y); free(h1);
    }
    return failed ? RRO_NOMEM : RRO_OK;
}

/*
 * Backward of one live row (token i at expert e with combine weight w):
 *   delta = <dout_i, y>           (what the weight's gradient sees)
 *   dy    = w dout_i
 *   dact  = W2_e^T dy
 *   dh3   = dact * silu(h1),  dh1 = dact * h3 * silu'(h1)
 *   dx    = W1_e^T dh1 + W3_e^T dh3
 * The gradient w.r.t. the hidden state flows through the experts only; the
 * gate projection a = W_g x is outside the layer (its caller owns dlogits).
 */
static double row_backward(const double *x, const double *dout, double w, const void *W1,
                           const void *W3, const void *W2, int e, int d, int d_ff, int dtype,
                           double *h1, double *h3, double *act, double *y, double *dh1,
                           double *dh3, double *dx_acc)
{
    size_t w13 = (size_t)e * d_ff * d, w2 = (size_t)e * d * d_ff;
    expert_forward(x, W1, W3, W2, e, d, d_ff, dtype, h1, h3, act, y);
    double delta = 0.0;
    for (int n = 0; n < d; ++n) delta += dout[n] * y[n];
    for (int f = 0; f < d_ff; ++f) {
        double dact = 0.0;
        for (int n = 0; n < d; ++n) dact += ld(W2, w2 + (size_t)n * d_ff + f, dtype) * (w * dout[n]);
        dh3[f] = dact * silu(h1[f]);
        dh1[f] = dact * h3[f] * dsilu(h1[f]);
    }
    if (dx_acc) {
        for (int c = 0; c < d; ++c) {
            double s = 0.0;
            for (int f = 0; f < d_ff; ++f)
                s += ld(W1, w13 + (size_t)f * d + c, dtype) * dh1[f] +
                     ld(W3, w13 + (size_t)f * d + c, dtype) * dh3[f];
            dx_acc[c] += s;
        }
    }
    return delta;
}

/*
 * rro_backward_tokens: for the listed tokens, dhidden_i [n_tok,d] and
 * dlogits_i [n_tok,E] (fp64), given dout [T,d].
 *
 * Gate gradient, two variants (Appendix A):
 *  exact (grad_exact != 0): differentiate w_r = mu_r e^{a_r} / sum mu e^{a}:
 *      dL/da_ij = sum_{r: e_r = j} w_r ( delta_r - sum_r' w_r' delta_r' ),
 *      zero for every expert outside the token's routes and identically zero
 *      when the token has a single route (the defect Appendix A describes).
 *  straight-through (default, Eq. 6): with g = softmax(a_i) over all E experts
 *      and S_i = sum_r mu_r g_{e_r} held constant,
 *      dL/dg_ij = sum_{r: e_r = j} mu_r delta_r / S_i, then through the full
 *      softmax: dL/da_il = g_il ( dL/dg_il - sum_j g_ij dL/dg_ij ).
 */
int rro_backward_tokens(const void *hidden, const void *W1, const void *W3, const void *W2,
                        const void *dout, int dtype, const float *logits, int T, int E, int k,
                        int d, int d_ff, int grad_exact, const int32_t *topk_expert,
                        const int32_t *route_slot, const int32_t *drop_count,
                        const int32_t *ir_expert, const int32_t *tokens, int n_tok,
                        double *dhidden, double *dlogits)
{
    if (k > 64) return RRO_INVALID;
    int failed = 0;
#pragma omp parallel
    {
        double *buf = (double *)malloc(sizeof(double) * ((size_t)d * 3 + (size_t)d_ff * 5 + 2 * (size_t)E));
        if (!buf) {
#pragma omp atomic write
            failed = 1;
        } else {
            double *x = buf, *y = x + d, *g_out = y + d;
            double *h1 = g_out + d, *h3 = h1 + d_ff, *act = h3 + d_ff, *dh1 = act + d_ff, *dh3 = dh1 + d_ff;
            double *g = dh3 + d_ff, *dLdg = g + E;
#pragma omp for schedule(dynamic, 1)
            for (int t = 0; t < n_tok; ++t) {
                int i = tokens[t];
                const float *a = logits + (size_t)i * E;
                const int32_t *sel = topk_expert + (size_t)i * (k + 1);
                const int32_t *slot = route_slot + (size_t)i * (k + 1);
                double w[64 + 2], delta[64 + 2], mu[64 + 2];
                token_weights(a, E, k, sel, slot, drop_count[i], ir_expert[i], w);
                for (int c = 0; c < d; ++c) {
                    x[c] = ld(hidden, (size_t)i * d + c, dtype);
                    g_out[c] = ld(dout, (size_t)i * d + c, dtype);
                }
                double *dx = dhidden + (size_t)t * d;
                for (int c = 0; c < d; ++c) dx[c] = 0.0;
                for (int r = 0; r < k + 2; ++r) {
                    int e = route_expert(k, sel, slot, ir_expert[i], r);
                    delta[r] = 0.0;
                    mu[r] = 0.0;
                    if (e < 0) continue;
                    mu[r] = (r == k + 1) ? (double)drop_count[i] : 1.0;
                    delta[r] = row_backward(x, g_out, w[r], W1, W3, W2, e, d, d_ff, dtype, h1, h3,
                                            act, y, dh1, dh3, dx);
                }
                double *dl = dlogits + (size_t)t * E;
                for (int j = 0; j < E; ++j) dl[j] = 0.0;
                if (grad_exact) {
                    double mean = 0.0;
                    for (int r = 0; r < k + 2; ++r) mean += w[r] * delta[r];
                    for (int r = 0; r < k + 2; ++r) {
                        int e = route_expert(k, sel, slot, ir_expert[i], r);
                        if (e >= 0) dl[e] += w[r] * (delta[r] - mean);
                    }
                } else {
                    double m = a[0], Z = 0.0, S = 0.0, dot = 0.0;
                    for (int j = 1; j < E; ++j) if ((double)a[j] > m) m = a[j];
                    for (int j = 0; j < E; ++j) { g[j] = exp((double)a[j] - m); Z += g[j]; }
                    for (int j = 0; j < E; ++j) { g[j] /= Z; dLdg[j] = 0.0; }
                    for (int r = 0; r < k + 2; ++r) {
                        int e = route_expert(k, sel, slot, ir_expert[i], r);
                        if (e >= 0) S += mu[r] * g[e];
                    }
                    if (S > 0.0) {
                        for (int r = 0; r < k + 2; ++r) {
                            int e = route_expert(k, sel, slot, ir_expert[i], r);
                            if (e >= 0) dLdg[e] += mu[r] * delta[r] / S;
                        }
                        for (int j = 0; j < E; ++j) dot += g[j] * dLdg[j];
                        for (int j = 0; j < E; ++j) dl[j] = g[j] * (dLdg[j] - dot);
                    }
                }
            }
        }
        free(buf);
    }
    return failed ? RRO_NOMEM : RRO_OK;
}

/*
 * rro_backward_expert: weight gradients of ONE expert e, summed over all of
 * its live rows (rows row_offset[e] .. row_offset[e+1]-1 of the row space):
 *   dW2_e += dy (x) act,  dW1_e += dh1 (x) x,  dW3_e += dh3 (x) x
 * Outputs fp64: dW1,dW3 [d_ff,d], dW2 [d,d_ff] (this expert only, zeroed here).
 */
int rro_backward_expert(const void *hidden, const void *W1, const void *W3, const void *W2,
                        const void *dout, int dtype, int e, int d, int d_ff,
                        const int32_t *row_offset, const int32_t *row_token,
                        const double *row_weight, double *dW1, double *dW3, double *dW2)
{
    int r0 = row_offset[e], r1 = row_offset[e + 1], n = r1 - r0;
    size_t n13 = (size_t)d_ff * d;
    for (size_t q = 0; q < n13; ++q) { dW1[q] = 0.0; dW3[q] = 0.0; dW2[q] = 0.0; }
    if (n <= 0) return RRO_OK;
    /* per-row quantities first (independent rows), then the sums in row order */
    double *X = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *DY = (double *)malloc(sizeof(double) * (size_t)n * d);
    double *ACT = (double *)malloc(sizeof(double) * (size_t)n * d_ff);
    double *DH1 = (double *)malloc(sizeof(double) * (size_t)n * d_ff);
    double *DH3 = (double *)malloc(sizeof(double) * (size_t)n * d_ff);
    int failed = (!X || !DY || !ACT || !DH1 || !DH3);
    if (!failed) {
#pragma omp parallel
        {
            double *tmp = (double *)malloc(sizeof(double) * ((size_t)d * 2 + (size_t)d_ff * 2));
            if (!tmp) {
#pragma omp atomic write
                failed = 1;
            } else {
                double *y = tmp, *g_out = y + d, *h1 = g_out + d, *h3 = h1 + d_ff;
#pragma omp for schedule(dynamic, 1)
                for (int q = 0; q < n; ++q) {
                    int i = row_token[r0 + q];
                    double w = row_weight[r0 + q];
                    double *x = X + (size_t)q * d;
                    for (int c = 0; c < d; ++c) {
                        x[c] = ld(hidden, (size_t)i * d + c, dtype);
                        g_out[c] = ld(dout, (size_t)i * d + c, dtype);
                        DY[(size_t)q * d + c] = w * g_out[c];
                    }
                    row_backward(x, g_out, w, W1, W3, W2, e, d, d_ff, dtype, h1, h3,
                                 ACT + (size_t)q * d_ff, y, DH1 + (size_t)q * d_ff,
                                 DH3 + (size_t)q * d_ff, NULL);
                }
            }
            free(tmp);
        }
    }
    if (!failed) {
#pragma omp parallel for schedule(static)
        for (int f = 0; f < d_ff; ++f) {
            for (int q = 0; q < n; ++q) {
                double a1 = DH1[(size_t)q * d_ff + f], a3 = DH3[(size_t)q * d_ff + f];
                const double *x = X + (size_t)q * d;
                for (int c = 0; c < d; ++c) {
                    dW1[(size_t)f * d + c] += a1 * x[c];
                    dW3[(size_t)f * d + c] += a3 * x[c];
                }
            }
        }
#pragma omp parallel for schedule(static)
        for (int nn = 0; nn < d; ++nn) {
            for (int q = 0; q < n; ++q) {
                double dy = DY[(size_t)q * d + nn];
                const double *act = ACT + (size_t)q * d_ff;
                for (int f = 0; f < d_ff; ++f) dW2[(size_t)nn * d_ff + f] += dy * act[f];
            }
        }
    }
    free(X); free(DY); free(ACT); free(DH1); free(DH3);
    return failed ? RRO_NOMEM : RRO_OK;
}

/*
 * rro_backward_expert_cols: the same sums as rro_backward_expert, restricted to a list of
 * FFN columns f (n_cols of them): rows f of dW1_e and dW3_e ([n_cols, d]) and columns f of
 * dW2_e ([d, n_cols]).  For a fixed f the quantities h1[f], h3[f], dact[f] of a row depend on no
 * other column, so every returned entry equals the corresponding entry of the full gradient;
 * this only makes full-size experts affordable.
 */
int rro_backward_expert_cols(const void *hidden, const void *W1, const void *W3, const void *W2,
                             const void *dout, int dtype, int e, int d, int d_ff,
                             const int32_t *row_offset, const int32_t *row_token,
                             const double *row_weight, const int32_t *cols, int n_cols,
                             double *dW1, double *dW3, double *dW2)
{
    int r0 = row_offset[e], r1 = row_offset[e + 1];
    size_t w13 = (size_t)e * d_ff * d, w2 = (size_t)e * d * d_ff;
#pragma omp parallel for schedule(dynamic, 1)
    for (int q = 0; q < n_cols; ++q) {
        int f = cols[q];
        double *g1 = dW1 + (size_t)q * d, *g3 = dW3 + (size_t)q * d;
        for (int c = 0; c < d; ++c) { g1[c] = 0.0; g3[c] = 0.0; dW2[(size_t)c * n_cols + q] = 0.0; }
        for (int r = r0; r < r1; ++r) {
            int i = row_token[r];
            double w = row_weight[r];
            double h1 = 0.0, h3 = 0.0, dact = 0.0;
            for (int c = 0; c < d; ++c) {
                double x = ld(hidden, (size_t)i * d + c, dtype);
                h1 += ld(W1, w13 + (size_t)f * d + c, dtype) * x;
                h3 += ld(W3, w13 + (size_t)f * d + c, dtype) * x;
                dact += ld(W2, w2 + (size_t)c * d_ff + f, dtype) * (w * ld(dout, (size_t)i * d + c, dtype));
            }
            double act = silu(h1) * h3;
            double dh3 = dact * silu(h1);
            double dh1 = dact * h3 * dsilu(h1);
            for (int c = 0; c < d; ++c) {
                double x = ld(hidden, (size_t)i * d + c, dtype);
                g1[c] += dh1 * x;
                g3[c] += dh3 * x;
                dW2[(size_t)c * n_cols + q] += (w * ld(dout, (size_t)i * d + c, dtype)) * act;
            }
        }
    }
    return RRO_OK;
}

/* ----------------------------------------------------------------------------
 * Gate projection (Section 3, Eq. 1): the score of token i at expert j is the
 * inner product of the expert's embedding vector with the token's hidden state,
 *     a_ij = w_j^T x_i.
 * Wg [E][d] holds the vectors w_j row by row.  fp64 sums of the exact input
 * values.                                                                    */
int rro_gate_fwd(const void *hidden, const void *Wg, int dtype, int T, int E, int d, double *logits)
{
    if (T < 0 || E < 1 || d < 1 || (dtype != RRO_F32 && dtype != RRO_BF16)) return RRO_INVALID;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < T; ++i)
        for (int j = 0; j < E; ++j) {
            double a = 0.0;
            for (int c = 0; c < d; ++c) a += ld(Wg, (size_t)j * d + c, dtype) * ld(hidden, (size_t)i * d + c, dtype);
            logits[(size_t)i * E + j] = a;
        }
    return RRO_OK;
}

/* Gradients of a loss L through a_ij = w_j^T x_i for given dL/da (the chain rule
 * on Eq. 1):  dL/dw_j = sum_i dL/da_ij x_i,   dL/dx_i (this path only) = sum_j dL/da_ij w_j. */
int rro_gate_bwd(const double *dlogits, const void *hidden, const void *Wg, int dtype, int T, int E, int d,
                 double *dWg, double *dhidden)
{
    if (T < 0 || E < 1 || d < 1 || (dtype != RRO_F32 && dtype != RRO_BF16)) return RRO_INVALID;
#pragma omp parallel for schedule(static)
    for (int j = 0; j < E; ++j)
        for (int c = 0; c < d; ++c) {
            double g = 0.0;
            for (int i = 0; i < T; ++i) g += dlogits[(size_t)i * E + j] * ld(hidden, (size_t)i * d + c, dtype);
            dWg[(size_t)j * d + c] = g;
        }
#pragma omp parallel for schedule(static)
    for (int i = 0; i < T; ++i)
        for (int c = 0; c < d; ++c) {
            double g = 0.0;
            for (int j = 0; j < E; ++j) g += dlogits[(size_t)i * E + j] * ld(Wg, (size_t)j * d + c, dtype);
            dhidden[(size_t)i * d + c] = g;
        }
    return RRO_OK;
}

/* ----------------------------------------------------------------------------
 * Load-balance loss of the top-k router (Section 5.1 gives its weight, 1e-2;
 * Appendix "Impact of Load-Balance Loss" names its source).  The paper prints no
 * formula; this is the one of the work it cites:
 *     f_e = (1/T) #{ i : first choice of token i is expert e }   (before capacity)
 *     P_e = (1/T) sum_i g_ie ,   g_i = softmax(a_i) over all E experts
 *     L   = alpha * E * sum_e f_e P_e .
 * first[i*stride] is the rank-0 expert of token i (column 0 of topk_expert).  */
int rro_aux_loss(const float *logits, const int32_t *first, int stride, int T, int E, double alpha,
                 double *loss, double *f, double *P)
{
    if (T < 1 || E < 1 || stride < 1) return RRO_INVALID;
    for (int e = 0; e < E; ++e) f[e] = P[e] = 0.0;
    for (int i = 0; i < T; ++i) {
        const float *a = logits + (size_t)i * E;
        int c = first[(size_t)i * stride];
        if (c < 0 || c >= E) return RRO_INVALID;
        f[c] += 1.0;
        double m = a[0], z = 0.0;
        for (int j = 1; j < E; ++j) if ((double)a[j] > m) m = a[j];
        for (int j = 0; j < E; ++j) z += exp((double)a[j] - m);
        for (int j = 0; j < E; ++j) P[j] += exp((double)a[j] - m) / z;
    }
    double acc = 0.0;
    for (int e = 0; e < E; ++e) { f[e] /= T; P[e] /= T; acc += f[e] * P[e]; }
    *loss = alpha * E * acc;
    return RRO_OK;
}

/* Gradient of that loss with the counts f held constant (they are piecewise constant in a):
 *     dL/da_ij = scale * alpha * E / T * g_ij * ( f_j - sum_e f_e g_ie ),
 * `scale` being dLoss/dL of whatever the caller adds L to.                    */
int rro_aux_loss_bwd(const float *logits, const double *f, int T, int E, double alpha, double scale,
                     double *dlogits)
{
    if (T < 1 || E < 1) return RRO_INVALID;
#pragma omp parallel for schedule(static)
    for (int i = 0; i < T; ++i) {
        const float *a = logits + (size_t)i * E;
        double m = a[0], z = 0.0, dot = 0.0;
        for (int j = 1; j < E; ++j) if ((double)a[j] > m) m = a[j];
        for (int j = 0; j < E; ++j) z += exp((double)a[j] - m);
        for (int j = 0; j < E; ++j) dot += f[j] * exp((double)a[j] - m) / z;
        for (int j = 0; j < E; ++j)
            dlogits[(size_t)i * E + j] = scale * alpha * E / T * (exp((double)a[j] - m) / z) * (f[j] - dot);
    }
    return RRO_OK;
}

/*
 * CPU oracle for Mixture-of-Contexts routing + sparse attention.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow, fp64.  It shares no code with the CUDA
 * library and is never called by it; only tests, the smoke check and the bench's
 * CPU-baseline leg may execute it.
 *
 * Conventions: H heads, L tokens, d head dim, C chunks.  Chunk c holds tokens
 * [off[c], off[c+1]); shot[c] is its shot id, mod[c] its modality (0 video, 1
 * text).  Q, K, V, dO are bf16 bit patterns (uint16) laid out [H][L][d]; every
 * value is widened exactly to double before use.
 *
 * Parity pins (tests/test_oracle_*.py): constant / ramp chunks for the descriptor;
 * enumeration of all k-subsets and a library top-k for the selection; the all-tie
 * case Q = 0 (first candidates win, LSE = log |selected tokens|); fp64 library
 * softmax attention with an explicit mask and its autograd for forward and
 * backward; finite differences; the paper's printed sparsity column for the pair
 * count; the published known-answer vectors for the counter-based generator and closed-form
 * expectations, set relations and the identity case for the drop-off / drop-in regulariser;
 * einsum and an independent numpy restatement for the shot-level (outer-loop) routing.
 * No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define MOC_ORACLE_WHOLE_SHOT (-1)

typedef struct {
    int H, L, d, C;
    int k;               /* routed picks per query (anchors not counted)            */
    int win_back;        /* intra-shot window, chunks before; -1 = the whole shot   */
    int win_fwd;         /* intra-shot window, chunks after;  -1 = the whole shot   */
    int causal;          /* 1: routed candidates are strictly earlier chunks        */
    const int32_t *off;  /* [C+1] */
    const int32_t *shot; /* [C]   */
    const uint8_t *mod;  /* [C]   */
} moc_oracle_cfg;

static inline double bf16_to_f64(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* chunk that holds token t (linear scan: obviously right, C is small) */
static int chunk_of(const moc_oracle_cfg *p, int t) {
    for (int c = 0; c < p->C; ++c)
        if (t >= p->off[c] && t < p->off[c + 1]) return c;
    return -1;
}

/* Sec. 3.2 "Fixed Cross-Modal Selection" + "Fixed Intra-Shot Selection": chunk j is a
 * mandatory anchor of a query living in chunk c if it is a text chunk, or if it lies
 * in c's shot within the window [c - win_back, c + win_fwd] (whole shot when -1). */
static int is_anchor(const moc_oracle_cfg *p, int c, int j) {
    if (p->mod[j] == 1) return 1;
    if (p->shot[j] != p->shot[c]) return 0;
    if (j < c && p->win_back != MOC_ORACLE_WHOLE_SHOT && c - j > p->win_back) return 0;
    if (j > c && p->win_fwd != MOC_ORACLE_WHOLE_SHOT && j - c > p->win_fwd) return 0;
    return 1;
}

/* Sec. 3.2 "Causality": an edge to chunk j >= c is masked before top-k; Sec. 3.3: forced
 * links are taken out of the candidate set before top-k. */
static int is_candidate(const moc_oracle_cfg *p, int c, int j) {
    if (is_anchor(p, c, j)) return 0;
    if (p->causal && j >= c) return 0;
    return 1;
}

/* ---- step 1: descriptors, Eq. 3 text: phi(K_w) = mean of the chunk's keys ---- */
void moc_oracle_chunk_pool(const moc_oracle_cfg *p, const uint16_t *K, double *desc /* [H][C][d] */) {
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int h = 0; h < p->H; ++h)
        for (int c = 0; c < p->C; ++c) {
            double *out = desc + ((size_t)h * p->C + c) * p->d;
            int n = p->off[c + 1] - p->off[c];
            for (int x = 0; x < p->d; ++x) {
                double s = 0.0;
                for (int t = p->off[c]; t < p->off[c + 1]; ++t)
                    s += bf16_to_f64(K[((size_t)h * p->L + t) * p->d + x]);
                out[x] = s / (double)n;
            }
        }
}

/* raw routing score of Eq. 3: q_i . phi_j (no 1/sqrt(d)) */
static double score(const moc_oracle_cfg *p, const uint16_t *Q, const double *desc, int h, int i, int j) {
    const uint16_t *q = Q + ((size_t)h * p->L + i) * p->d;
    const double *f = desc + ((size_t)h * p->C + j) * p->d;
    double s = 0.0;
    for (int x = 0; x < p->d; ++x) s += bf16_to_f64(q[x]) * f[x];
    return s;
}

/* scores of given rows against all chunks: out[n][C] (no masking) */
void moc_oracle_scores(const moc_oracle_cfg *p, const uint16_t *Q, const double *desc, int n,
                       const int32_t *rows /* [n][2] = (h, i) */, double *out) {
#pragma omp parallel for schedule(dynamic, 16)
    for (int r = 0; r < n; ++r)
        for (int j = 0; j < p->C; ++j)
            out[(size_t)r * p->C + j] = score(p, Q, desc, rows[2 * r], rows[2 * r + 1], j);
}

/* ---- steps 2-5 for one query: the k best candidates, one at a time; among equal
 * scores the lower chunk index wins.  sel gets k entries, -1 padded. ---- */
static void route_row(const moc_oracle_cfg *p, const uint16_t *Q, const double *desc, int h, int i,
                      int32_t *sel, double *sel_score, double *next_score) {
    int C = p->C, c = chunk_of(p, i);
    double *s = (double *)malloc(sizeof(double) * C);
    char *avail = (char *)malloc(C);
    for (int j = 0; j < C; ++j) {
        avail[j] = (char)is_candidate(p, c, j);
        s[j] = avail[j] ? score(p, Q, desc, h, i, j) : 0.0;
    }
    for (int r = 0; r <= p->k; ++r) {
        int best = -1;
        for (int j = 0; j < C; ++j)
            if (avail[j] && (best < 0 || s[j] > s[best])) best = j; /* strict >: lower index wins ties */
        if (r == p->k) { /* best candidate left unselected, for near-tie bookkeeping */
            if (next_score) *next_score = best >= 0 ? s[best] : -INFINITY;
            break;
        }
        sel[r] = best;
        if (sel_score) sel_score[r] = best >= 0 ? s[best] : -INFINITY;
        if (best >= 0) avail[best] = 0;
    }
    free(s);
    free(avail);
}

void moc_oracle_route(const moc_oracle_cfg *p, const uint16_t *Q, const double *desc,
                      int32_t *sel_idx /* [H][L][k] */, double *sel_score /* [H][L][k] or NULL */,
                      double *next_score /* [H][L] or NULL */) {
#pragma omp parallel for collapse(2) schedule(dynamic, 64)
    for (int h = 0; h < p->H; ++h)
        for (int i = 0; i < p->L; ++i) {
            size_t r = (size_t)h * p->L + i;
            route_row(p, Q, desc, h, i, sel_idx + r * p->k, sel_score ? sel_score + r * p->k : NULL,
                      next_score ? next_score + r : NULL);
        }
}

/* ---- step 6: explicit token mask of one query: Omega = anchors U routed picks ---- */
static void token_mask_row(const moc_oracle_cfg *p, int i, const int32_t *sel, uint8_t *mask /* [L] */) {
    int c = chunk_of(p, i);
    memset(mask, 0, (size_t)p->L);
    for (int j = 0; j < p->C; ++j) {
        int on = is_anchor(p, c, j);
        for (int r = 0; r < p->k && !on; ++r) on = (sel[r] == j);
        if (on)
            for (int t = p->off[j]; t < p->off[j + 1]; ++t) mask[t] = 1;
    }
}

void moc_oracle_token_mask(const moc_oracle_cfg *p, int i, const int32_t *sel, uint8_t *mask) {
    token_mask_row(p, i, sel, mask);
}

/* number of selected (query, key) pairs of given rows, from the explicit masks */
int64_t moc_oracle_pair_count(const moc_oracle_cfg *p, const int32_t *sel_idx, int n, const int32_t *rows) {
    int64_t total = 0;
#pragma omp parallel reduction(+ : total)
    {
        uint8_t *mask = (uint8_t *)malloc((size_t)p->L);
#pragma omp for schedule(dynamic, 16)
        for (int r = 0; r < n; ++r) {
            int h = rows[2 * r], i = rows[2 * r + 1];
            token_mask_row(p, i, sel_idx + ((size_t)h * p->L + i) * p->k, mask);
            for (int t = 0; t < p->L; ++t) total += mask[t];
        }
        free(mask);
    }
    return total;
}

/* ---- step 7 for one query: masked dense softmax attention, Eq. 2 / Eq. 1.
 * prob (optional, [L]) receives P_it (0 off the mask). ---- */
static void attend_row(const moc_oracle_cfg *p, const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                       int h, int i, const uint8_t *mask, double scale, double *o /* [d] */, double *lse,
                       double *prob, double *z /* scratch [L] */) {
    int d = p->d, L = p->L;
    const uint16_t *q = Q + ((size_t)h * L + i) * d;
    double zmax = -INFINITY;
    for (int t = 0; t < L; ++t) {
        if (!mask[t]) continue;
        const uint16_t *kt = K + ((size_t)h * L + t) * d;
        double s = 0.0;
        for (int x = 0; x < d; ++x) s += bf16_to_f64(q[x]) * bf16_to_f64(kt[x]);
        z[t] = s * scale;
        if (z[t] > zmax) zmax = z[t];
    }
    double den = 0.0;
    for (int t = 0; t < L; ++t)
        if (mask[t]) den += exp(z[t] - zmax);
    *lse = zmax + log(den);
    for (int x = 0; x < d; ++x) o[x] = 0.0;
    for (int t = 0; t < L; ++t) {
        double pt = mask[t] ? exp(z[t] - *lse) : 0.0;
        if (prob) prob[t] = pt;
        if (!mask[t]) continue;
        const uint16_t *vt = V + ((size_t)h * L + t) * d;
        for (int x = 0; x < d; ++x) o[x] += pt * bf16_to_f64(vt[x]);
    }
}

static double default_scale(const moc_oracle_cfg *p, double scale) {
    return scale > 0.0 ? scale : 1.0 / sqrt((double)p->d);
}

/* forward of given rows: O [n][d], lse [n] */
void moc_oracle_attend_rows(const moc_oracle_cfg *p, const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                            const int32_t *sel_idx, double scale, int n, const int32_t *rows, double *O,
                            double *lse) {
    scale = default_scale(p, scale);
#pragma omp parallel
    {
        uint8_t *mask = (uint8_t *)malloc((size_t)p->L);
        double *z = (double *)malloc(sizeof(double) * (size_t)p->L);
#pragma omp for schedule(dynamic, 4)
        for (int r = 0; r < n; ++r) {
            int h = rows[2 * r], i = rows[2 * r + 1];
            token_mask_row(p, i, sel_idx + ((size_t)h * p->L + i) * p->k, mask);
            attend_row(p, Q, K, V, h, i, mask, scale, O + (size_t)r * p->d, lse + r, NULL, z);
        }
        free(mask);
        free(z);
    }
}

/* ---- step 8: backward with the mask held constant (Sec. 3.1: top-k is not
 * differentiated; gradients reach Q, K, V only through the selected attention).
 *   D_i = dO_i . O_i;  dV_t = sum_i P_it dO_i;  dS_it = P_it (dO_i . v_t - D_i);
 *   dQ_i = scale sum_t dS_it k_t;  dK_t = scale sum_i dS_it q_i.
 * dQ is returned for the listed rows ([n][d]); dK, dV for tokens [t0, t1) of head
 * key_head ([t1-t0][d]), summed over EVERY query of that head whose mask reaches them
 * (each such query's forward is recomputed).  Pass n = 0 or t1 <= t0 to skip a part. */
void moc_oracle_attend_bwd(const moc_oracle_cfg *p, const uint16_t *Q, const uint16_t *K, const uint16_t *V,
                           const uint16_t *dO, const int32_t *sel_idx, double scale, int n, const int32_t *rows,
                           double *dQ, int key_head, int t0, int t1, double *dK, double *dV) {
    int d = p->d, L = p->L;
    scale = default_scale(p, scale);
    int nk = t1 > t0 ? t1 - t0 : 0;
    if (nk > 0) {
        memset(dK, 0, sizeof(double) * (size_t)nk * d);
        memset(dV, 0, sizeof(double) * (size_t)nk * d);
    }
    int total = n + (nk > 0 ? L : 0); /* work items: listed rows, then every query of key_head */
#pragma omp parallel
    {
        uint8_t *mask = (uint8_t *)malloc((size_t)L);
        double *z = (double *)malloc(sizeof(double) * (size_t)L);
        double *prob = (double *)malloc(sizeof(double) * (size_t)L);
        double *o = (double *)malloc(sizeof(double) * d);
        double *aK = nk > 0 ? (double *)calloc((size_t)nk * d, sizeof(double)) : NULL;
        double *aV = nk > 0 ? (double *)calloc((size_t)nk * d, sizeof(double)) : NULL;
#pragma omp for schedule(dynamic, 4)
        for (int w = 0; w < total; ++w) {
            int for_q = w < n;
            int h = for_q ? rows[2 * w] : key_head;
            int i = for_q ? rows[2 * w + 1] : w - n;
            token_mask_row(p, i, sel_idx + ((size_t)h * L + i) * p->k, mask);
            if (!for_q) {
                int hit = 0;
                for (int t = t0; t < t1 && !hit; ++t) hit = mask[t];
                if (!hit) continue;
            }
            double lse;
            attend_row(p, Q, K, V, h, i, mask, scale, o, &lse, prob, z);
            const uint16_t *doi = dO + ((size_t)h * L + i) * d;
            const uint16_t *qi = Q + ((size_t)h * L + i) * d;
            double D = 0.0;
            for (int x = 0; x < d; ++x) D += bf16_to_f64(doi[x]) * o[x];
            if (for_q) {
                double *dq = dQ + (size_t)w * d;
                for (int x = 0; x < d; ++x) dq[x] = 0.0;
                for (int t = 0; t < L; ++t) {
                    if (!mask[t]) continue;
                    const uint16_t *vt = V + ((size_t)h * L + t) * d;
                    const uint16_t *kt = K + ((size_t)h * L + t) * d;
                    double dp = 0.0;
                    for (int x = 0; x < d; ++x) dp += bf16_to_f64(doi[x]) * bf16_to_f64(vt[x]);
                    double ds = prob[t] * (dp - D);
                    for (int x = 0; x < d; ++x) dq[x] += scale * ds * bf16_to_f64(kt[x]);
                }
            } else {
                for (int t = t0; t < t1; ++t) {
                    if (!mask[t]) continue;
                    const uint16_t *vt = V + ((size_t)h * L + t) * d;
                    double dp = 0.0;
                    for (int x = 0; x < d; ++x) dp += bf16_to_f64(doi[x]) * bf16_to_f64(vt[x]);
                    double ds = prob[t] * (dp - D);
                    double *ak = aK + (size_t)(t - t0) * d, *av = aV + (size_t)(t - t0) * d;
                    for (int x = 0; x < d; ++x) {
                        av[x] += prob[t] * bf16_to_f64(doi[x]);
                        ak[x] += scale * ds * bf16_to_f64(qi[x]);
                    }
                }
            }
        }
        if (nk > 0) {
#pragma omp critical
            for (size_t e = 0; e < (size_t)nk * d; ++e) {
                dK[e] += aK[e];
                dV[e] += aV[e];
            }
        }
        free(mask); free(z); free(prob); free(o); free(aK); free(aV);
    }
}


/* ---- Counter-based random numbers: Philox4x32-10 as defined by Salmon, Moraes, Dror and Shaw,
 * "Parallel random numbers: as easy as 1, 2, 3" (SC'11): ten rounds of
 *   (c0, c1, c2, c3) <- (hi(M1 c2) ^ c1 ^ k0,  lo(M1 c2),  hi(M0 c0) ^ c3 ^ k1,  lo(M0 c0))
 * with M0 = 0xD2511F53, M1 = 0xCD9E8D57, the key bumped by (0x9E3779B9, 0xBB67AE85) between rounds.
 * The regulariser below draws from it; the CUDA library has its own implementation of the same
 * definition.  Pinned by the known-answer vectors published with the generator. ---- */
void moc_oracle_philox4x32(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0, p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* d-th uniform draw of row (h, i): word d % 4 of the block with counter (i, h, d / 4, 0) and key = seed;
 * its top 24 bits scaled to [0, 1), which is exact in single precision. */
static float row_uniform(uint64_t seed, int h, int i, int d) {
    uint32_t ctr[4] = {(uint32_t)i, (uint32_t)h, (uint32_t)(d / 4), 0u}, key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)}, out[4];
    moc_oracle_philox4x32(ctr, key, out);
    return (float)(out[d % 4] >> 8) * (1.0f / 16777216.0f);
}

/* ---- Sec. 3.1 "Context drop-off" and "Context drop-in": training-time edits of a routed selection.
 * For every query (h, i), on its k slots (the paper's top-k; -1 = empty slot):
 *   drop-off: p_drop = U * p_max with U ~ Uniform[0, 1); floor(p_drop * k) of the row's picks (never more
 *             than it has) are removed, each chosen uniformly among the picks still there;
 *   drop-in:  m ~ Poisson(lambda) chunks are added, each chosen uniformly among the chunks that may be
 *             routed to from the row (not an anchor, strictly earlier if causal) and that are neither in the
 *             routed selection nor added already; they go into the free slots (empty or just dropped),
 *             lowest slot first, for as long as there is a free slot and a chunk left to add.
 * Where a draw decides an integer the arithmetic is single precision, as in the CUDA kernel:
 *   draw 0: U;  draw 1: the Poisson variate by inversion (smallest m with u < cdf[m], cdf accumulated in
 *   double from exp(-lambda) by term_j = term_{j-1} lambda / j and rounded to single; at most 31);
 *   draw 2 + r: the r-th removal takes the floor(u * n_left)-th pick still there, in slot order;
 *   draw 2 + k + t: the t-th addition takes the floor(u * n_left)-th eligible chunk, in chunk order.
 * n_dropped / n_drawn / n_added ([H][L], optional) report what happened per row. ---- */
void moc_oracle_context_drop(const moc_oracle_cfg *p, int32_t *sel_idx, float p_max, float lambda, uint64_t seed,
                             int32_t *n_dropped, int32_t *n_drawn, int32_t *n_added) {
    float cdf[32];
    {
        double term = exp(-(double)lambda), acc = term;
        cdf[0] = (float)acc;
        for (int j = 1; j < 32; ++j) {
            term = term * (double)lambda / (double)j;
            acc += term;
            cdf[j] = (float)acc;
        }
    }
    int k = p->k;
#pragma omp parallel for collapse(2) schedule(dynamic, 64)
    for (int h = 0; h < p->H; ++h)
        for (int i = 0; i < p->L; ++i) {
            int32_t *row = sel_idx + ((size_t)h * p->L + i) * k;
            int c = chunk_of(p, i);
            int32_t *orig = (int32_t *)malloc(sizeof(int32_t) * (size_t)(k > 0 ? k : 1));
            char *gone = (char *)calloc((size_t)(k > 0 ? k : 1), 1);       /* 1: this slot's pick was dropped */
            memcpy(orig, row, sizeof(int32_t) * (size_t)k);
            int n_sel = 0;
            for (int s = 0; s < k; ++s) n_sel += orig[s] >= 0;
            /* drop-off */
            float p_drop = row_uniform(seed, h, i, 0) * p_max;
            int n_drop = (int)(p_drop * (float)k);
            if (n_drop > n_sel) n_drop = n_sel;
            for (int r = 0; r < n_drop; ++r) {
                int n_left = n_sel - r;
                int pos = (int)(row_uniform(seed, h, i, 2 + r) * (float)n_left);
                if (pos > n_left - 1) pos = n_left - 1;
                for (int s = 0; s < k; ++s) {
                    if (orig[s] < 0 || gone[s]) continue;
                    if (pos-- == 0) { gone[s] = 1; row[s] = -1; break; }
                }
            }
            /* drop-in */
            float u = row_uniform(seed, h, i, 1);
            int m = 0;
            while (m < 31 && !(u < cdf[m])) ++m;
            int added = 0;
            for (int t = 0; t < m; ++t) {
                int slot = -1;
                for (int s = 0; s < k && slot < 0; ++s)
                    if (row[s] < 0) slot = s;
                if (slot < 0) break;
                /* eligible: a candidate of the row that is neither a routed pick (kept or dropped) nor added already */
                int n_left = 0;
                for (int j = 0; j < p->C; ++j) {
                    if (!is_candidate(p, c, j)) continue;
                    int used = 0;
                    for (int s = 0; s < k && !used; ++s) used = (orig[s] == j) || (row[s] == j);
                    n_left += !used;
                }
                if (n_left == 0) break;
                int pos = (int)(row_uniform(seed, h, i, 2 + k + t) * (float)n_left);
                if (pos > n_left - 1) pos = n_left - 1;
                for (int j = 0; j < p->C; ++j) {
                    if (!is_candidate(p, c, j)) continue;
                    int used = 0;
                    for (int s = 0; s < k && !used; ++s) used = (orig[s] == j) || (row[s] == j);
                    if (used) continue;
                    if (pos-- == 0) { row[slot] = j; break; }
                }
                ++added;
            }
            size_t r_ = (size_t)h * p->L + i;
            if (n_dropped) n_dropped[r_] = n_drop;
            if (n_drawn) n_drawn[r_] = m;
            if (n_added) n_added[r_] = added;
            free(orig);
            free(gone);
        }
}


/* ---- Appendix "Outer Loop Context Routing": a coarse pre-selection of whole shots for one query block.
 * High-level chunk Psi_s = every token of shot s (all of its chunks, in stream order).  Per feature stream h:
 *   phi(Psi_s) = mean of Xk over the tokens of shot s;   x_g = mean of Xq over the query block [q0, q1);
 *   s_s = <x_g, phi(Psi_s)>;   Omega_g = the M shots of largest s_s among the shots that END before the block
 *   begins (a shot holding a token >= q0 is the block's own present or future and is not a candidate); equal
 *   scores go to the earlier shot; fewer than M candidates: all of them, -1 padded.
 * shot_desc [H][S][d], scores [H][S] (every shot, unmasked), sel [H][M]; S = number of distinct shot ids. ---- */
int moc_oracle_num_shots(const moc_oracle_cfg *p) {
    int S = 0;
    for (int c = 0; c < p->C; ++c)
        if (c == 0 || p->shot[c] != p->shot[c - 1]) ++S;
    return S;
}

void moc_oracle_outer_route(const moc_oracle_cfg *p, const uint16_t *Xq, const uint16_t *Xk, int q0, int q1, int M,
                            double *shot_desc, double *scores, int32_t *sel) {
    int S = moc_oracle_num_shots(p), d = p->d, L = p->L;
    int *t0 = (int *)malloc(sizeof(int) * (size_t)S), *t1 = (int *)malloc(sizeof(int) * (size_t)S);
    for (int c = 0, s = -1; c < p->C; ++c) {
        if (c == 0 || p->shot[c] != p->shot[c - 1]) { ++s; t0[s] = p->off[c]; }
        t1[s] = p->off[c + 1];
    }
    for (int h = 0; h < p->H; ++h) {
        double *xg = (double *)calloc((size_t)d, sizeof(double));
        for (int t = q0; t < q1; ++t)
            for (int x = 0; x < d; ++x) xg[x] += bf16_to_f64(Xq[((size_t)h * L + t) * d + x]);
        for (int x = 0; x < d; ++x) xg[x] /= (double)(q1 - q0);
        for (int s = 0; s < S; ++s) {
            double *f = shot_desc + ((size_t)h * S + s) * d;
            for (int x = 0; x < d; ++x) {
                double a = 0.0;
                for (int t = t0[s]; t < t1[s]; ++t) a += bf16_to_f64(Xk[((size_t)h * L + t) * d + x]);
                f[x] = a / (double)(t1[s] - t0[s]);
            }
            double sc = 0.0;
            for (int x = 0; x < d; ++x) sc += xg[x] * f[x];
            scores[(size_t)h * S + s] = sc;
        }
        char *avail = (char *)malloc((size_t)S);
        for (int s = 0; s < S; ++s) avail[s] = (char)(t1[s] <= q0);
        for (int r = 0; r < M; ++r) {
            int best = -1;
            for (int s = 0; s < S; ++s)
                if (avail[s] && (best < 0 || scores[(size_t)h * S + s] > scores[(size_t)h * S + best])) best = s;
            sel[(size_t)h * M + r] = best;
            if (best >= 0) avail[best] = 0;
        }
        free(avail);
        free(xg);
    }
    free(t0);
    free(t1);
}

int moc_oracle_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    n = omp_get_max_threads();
#endif
    return n;
}

/*
 * CPU oracle for the CASK compression event -- TEST INFRASTRUCTURE ONLY.
 *
 * A plain, slow, double-precision restatement of what one compression event
 * computes for one unit (one sequence x layer x KV head).  It is used by the
 * tests, the smoke check and the benchmark's cpu_baseline leg to judge the
 * CUDA library; it shares no code with that library and the library never
 * calls it.  No blocking, fusion or reordering: every function walks the
 * definition it cites so it can be checked against the paper by eye.
 *
 * Where the paper states a formula the function cites it.  Where the paper is
 * silent the reading taken here is listed beside the function ("reading:");
 * those choices (score form, gamma, tau, eps, reserve, seed rule) are fixed by
 * this project's written definition, not by the paper: for them parity with
 * the paper itself is "parity unpinned".
 *
 * Inputs are the cache values as float (bf16 or fp32 values, promoted exactly
 * to double).  Row kinds: 0 dropped, 1 kept prefix, 2 recent, 3 core, 4 seed
 * (representative anchor), 5 merged into a seed's group.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum {
    ORC_NOOP_UNDER_BUDGET = 1,
    ORC_PREFIX_EVICTED = 2,
    ORC_DECODE_CONSOLIDATED = 4,
    ORC_PREFIX_BUDGET_EXHAUSTED = 8,
    ORC_MERGE_INACTIVE = 16
};

enum { PL_BP = 0, PL_PKEEP, PL_BD, PL_R, PL_C, PL_M, PL_FLAGS, PL_NOUT };

/*
 * Merge weight of a row (Sec. 2.4 leaves a_i open: "local score mass, similarity weight, or
 * position-aware importance").  Reading: a_i = s_i + eps, plus the group mass the row already
 * carries when it is itself a representative of an earlier event (mass_in, nullable), so that
 * folding "preserves group mass" across events.
 */
static double orc_a(const double* s, const double* mass_in, double eps, int i) {
    return s[i] + eps + (mass_in ? mass_in[i] : 0.0);
}

/* ---- total order used by every selection: score descending, row ascending ---- */
typedef struct { double s; int i; } orc_item;

static int orc_cmp(const void* a, const void* b) {
    const orc_item* x = (const orc_item*)a;
    const orc_item* y = (const orc_item*)b;
    if (x->s > y->s) return -1;
    if (x->s < y->s) return 1;
    return (x->i > y->i) - (x->i < y->i);
}

/*
 * Score (Sec. 1 "assign scalar importance to each token"; the deployed scorer
 * has no formula in the paper -- reading: windowed attention mass).
 * For query head h < g and window position j < W, with the window query j
 * sitting at cache row T-W+j:
 *     x_hji = <q_hj, k_i> / sqrt(d)
 *     key i is visible to query j  iff  i <= T-W+j      (causal != 0; else all)
 *     lse_hj = log sum_{visible i} exp(x_hji)
 *     p_hji  = exp(x_hji - lse_hj) on visible keys, 0 elsewhere
 *     s_i    = (1/(g W)) sum_{h,j} p_hji
 * lse_in (nullable, [g*W]) replaces the computed normaliser.
 */
void cask_oracle_score(const float* K, const float* Q, int T, int d, int g, int W, int causal,
                       const double* lse_in, double* s, double* lse_out) {
    double* x = (double*)malloc(sizeof(double) * (size_t)(T > 0 ? T : 1));
    const double inv_sqrt_d = 1.0 / sqrt((double)d);
    for (int i = 0; i < T; ++i) s[i] = 0.0;
    for (int h = 0; h < g; ++h) {
        for (int j = 0; j < W; ++j) {
            const float* q = Q + ((size_t)h * W + j) * d;
            int nvis = causal ? (T - W + j + 1) : T;
            if (nvis > T) nvis = T;
            if (nvis < 0) nvis = 0;
            double mx = -INFINITY;
            for (int i = 0; i < nvis; ++i) {
                const float* k = K + (size_t)i * d;
                double acc = 0.0;
                for (int c = 0; c < d; ++c) acc += (double)q[c] * (double)k[c];
                x[i] = acc * inv_sqrt_d;
                if (x[i] > mx) mx = x[i];
            }
            double lse;
            if (lse_in) {
                lse = lse_in[h * W + j];
            } else {
                double z = 0.0;
                for (int i = 0; i < nvis; ++i) z += exp(x[i] - mx);
                lse = (nvis > 0) ? mx + log(z) : 0.0;
            }
            if (lse_out) lse_out[h * W + j] = lse;
            for (int i = 0; i < nvis; ++i) s[i] += exp(x[i] - lse);
        }
    }
    const double inv_rows = 1.0 / ((double)g * (double)W);
    for (int i = 0; i < T; ++i) s[i] *= inv_rows;
    free(x);
}

/*
 * Budget split (Sec. 2.2: Stage 1 evicts the prefix "to secure slack for the
 * decode stage"; Sec. 2.3: |R| <= B, C subset of R, scratch uses only the
 * remaining budget; Sec. 5.2: when the prefix encroaches on the budget the
 * available slots collapse).  Reading (the paper gives no numbers):
 *   B_p = B - reserve;  P_keep = min(P, B_p);  B_d = B - P_keep;  N_d = T - P
 *   T <= B            -> NOOP_UNDER_BUDGET: every row kept
 *   r = min(W, N_d)      recent rows, always protected
 *   N_d <= B_d        -> every decode row kept as a singleton, no merge
 *   B_d < r + 2       -> PREFIX_BUDGET_EXHAUSTED: no room for the recent window
 *                        plus one core slot plus one representative; keep the
 *                        last min(r,B_d) rows and the best of the rest, no merge
 *   else c = min(ceil(gamma (B_d - r)), B_d - r - 1),  m = B_d - r - c  (>= 1)
 */
void cask_oracle_plan(int T, int P, int B, int reserve, int W, double gamma, int* plan) {
    int Nd = T - P;
    int Bp = B - reserve;
    int Pkeep = P < Bp ? P : Bp;
    int Bd = B - Pkeep;
    int r = W < Nd ? W : Nd;
    int c = 0, m = 0, flags = 0, nout;
    if (T <= B) {
        flags = ORC_NOOP_UNDER_BUDGET;
        Pkeep = P;
        Bd = B - P;
        c = Nd - r;
        nout = T;
    } else {
        if (P > Bp) flags |= ORC_PREFIX_EVICTED;
        if (Nd <= Bd) {
            c = Nd - r;
            nout = Pkeep + Nd;
        } else if (Bd < r + 2) {
            flags |= ORC_PREFIX_BUDGET_EXHAUSTED;
            r = r < Bd ? r : Bd;
            c = Bd - r;
            nout = Pkeep + Bd;
        } else {
            flags |= ORC_DECODE_CONSOLIDATED;
            int room = Bd - r;
            c = (int)ceil(gamma * (double)room);
            if (c > room - 1) c = room - 1;
            if (c < 0) c = 0;
            m = room - c;
            nout = Pkeep + Bd;
        }
    }
    plan[PL_BP] = Bp; plan[PL_PKEEP] = Pkeep; plan[PL_BD] = Bd; plan[PL_R] = r;
    plan[PL_C] = c; plan[PL_M] = m; plan[PL_FLAGS] = flags; plan[PL_NOUT] = nout;
}

/* mark the `k` greatest rows of [lo,hi) whose kind is 0 with `mark` */
static void orc_mark_top(const double* s, int lo, int hi, int k, uint8_t* kind, uint8_t mark) {
    int n = 0;
    orc_item* it = (orc_item*)malloc(sizeof(orc_item) * (size_t)(hi > lo ? hi - lo : 1));
    for (int i = lo; i < hi; ++i)
        if (kind[i] == 0) { it[n].s = s[i]; it[n].i = i; ++n; }
    qsort(it, (size_t)n, sizeof(orc_item), orc_cmp);
    if (k > n) k = n;
    for (int t = 0; t < k; ++t) kind[it[t].i] = mark;
    free(it);
}

/*
 * Stage 1, prefix eviction (Sec. 2.2).  If the prefix exceeds its share keep
 * its P_keep greatest rows under the total order; otherwise keep all of it.
 * Writes kind[0:P] (1 kept, 0 evicted).
 */
void cask_oracle_prefix_evict(const double* s, int P, const int* plan, uint8_t* kind) {
    for (int i = 0; i < P; ++i) kind[i] = 0;
    if (P <= plan[PL_PKEEP]) {
        for (int i = 0; i < P; ++i) kind[i] = 1;
    } else {
        orc_mark_top(s, 0, P, plan[PL_PKEEP], kind, 1);
    }
}

/*
 * Protected core (Sec. 2.1: answer formation / state anchoring -> highest
 * score; "recent reasoning pivots" -> recency).  recent = rows [T-r, T);
 * core = the c greatest rows of [P, T-r).  Writes kind[P:T] (2, 3, else 0).
 */
void cask_oracle_select_core(const double* s, int T, int P, const int* plan, uint8_t* kind) {
    int r = plan[PL_R], c = plan[PL_C];
    for (int i = P; i < T; ++i) kind[i] = 0;
    for (int i = T - r; i < T; ++i) kind[i] = 2;
    orc_mark_top(s, P, T - r, c, kind, 3);
}

/*
 * Kappa-weighted merge geometry in its own form (Sec. 2.5):
 *     d_kappa(k_i, k_j) = sum_f w_f * || k_{i,f} - k_{j,f} ||_2 ,   w_f = |kappa(omega_f)| >= 0 (caller-supplied),
 * where band f is a pair of channels of the rotary embedding: (f, f + d/2) for layout 0 (the halves of the head
 * are rotated against each other), (2f, 2f + 1) for layout 1 (adjacent channels).  The paper gives the distance
 * and no rule for turning it into a merge decision; reading: the scale-free similarity
 *     sim_kappa(j,u) = 1 - d_kappa(k_j,k_u) / (D_j + D_u),   D_x = sum_f w_f ||k_{x,f}||_2 ,
 * which lies in [0,1] by the triangle inequality (1 for equal keys, 0 for opposite ones), takes the place of the
 * cosine: argmax over the seeds, threshold tau, the same tie rule; a row or seed with D = 0 has similarity 0.
 */
static void orc_band(int f, int d, int layout, int* c0, int* c1) {
    if (layout == 0) { *c0 = f; *c1 = f + d / 2; }
    else { *c0 = 2 * f; *c1 = 2 * f + 1; }
}
static double orc_band_len(const float* k, int d, const float* bw, int layout) {
    double D = 0.0;
    for (int f = 0; f < d / 2; ++f) {
        int c0, c1;
        orc_band(f, d, layout, &c0, &c1);
        D += (double)bw[f] * sqrt((double)k[c0] * (double)k[c0] + (double)k[c1] * (double)k[c1]);
    }
    return D;
}
static double orc_band_dist(const float* a, const float* b, int d, const float* bw, int layout) {
    double dist = 0.0;
    for (int f = 0; f < d / 2; ++f) {
        int c0, c1;
        orc_band(f, d, layout, &c0, &c1);
        double x = (double)a[c0] - (double)b[c0], y = (double)a[c1] - (double)b[c1];
        dist += (double)bw[f] * sqrt(x * x + y * y);
    }
    return dist;
}

/*
 * Scratch consolidation (Sec. 2.1 "representative construction only on this
 * part"; Sec. 2.4 m-folding; Sec. 2.5 cosine as the base merge geometry).
 * Scratch S = rows of [P, T-r) with kind 0.  Reading: the m greatest rows of S
 * become seeds; every other j in S goes to the seed with the largest cosine
 * similarity of keys (ties: smallest seed row; a zero-norm row has similarity
 * 0) if that similarity is >= tau, else it is dropped and its a_j counts as
 * lost mass (the |Delta m_G| term of Sec. 2.6).  Merge weights (Sec. 2.4):
 *     a_i = s_i + eps (+ carried mass, see orc_a),  m_G = sum_{i in G} a_i,  w_i = a_i / m_G.
 * chan_w (nullable, [d], >= 0) weighs the channels of the similarity (Sec. 2.5: differences in frequency
 * bands with more future relevance count more; reading: the inner-product form
 *     sim_w(j,u) = sum_c w_c k_jc k_uc / (|k_j|_w |k_u|_w),  |k|_w^2 = sum_c w_c k_c^2,
 * with w_c = |kappa(omega_f)| on the channels of band f supplied by the caller; NULL = plain cosine).
 * band_w (nullable, [d/2], >= 0; not together with chan_w) selects the un-squared per-band form sim_kappa above.
 * Outputs: kind (adds 4 seed, 5 merged), seed_of (row of the group's seed, -1),
 * weight (w_i for group members, untouched elsewhere), sim / sim2 (best and
 * second-best similarity of each non-seed scratch row; -2 where undefined).
 * Returns flags to OR into the unit's status (MERGE_INACTIVE if nobody joins).
 */
int cask_oracle_consolidate(const float* K, const double* s, int T, int P, int d, const int* plan,
                            double tau, double eps, const double* mass_in, const float* chan_w,
                            const float* band_w, int band_layout, uint8_t* kind, int* seed_of,
                            double* weight, double* sim, double* sim2, double* lost_mass) {
    int r = plan[PL_R], m = plan[PL_M];
    for (int i = 0; i < T; ++i) { seed_of[i] = -1; if (sim) sim[i] = -2.0; if (sim2) sim2[i] = -2.0; }
    *lost_mass = 0.0;
    if (m <= 0) return 0;
    orc_mark_top(s, P, T - r, m, kind, 4);
    int* seeds = (int*)malloc(sizeof(int) * (size_t)m);
    double* snorm = (double*)malloc(sizeof(double) * (size_t)m);
    int ns = 0;
    for (int i = P; i < T - r; ++i)
        if (kind[i] == 4) {
            seeds[ns] = i;
            double n2 = 0.0;
            for (int c = 0; c < d; ++c)
                n2 += (chan_w ? (double)chan_w[c] : 1.0) * (double)K[(size_t)i * d + c] * (double)K[(size_t)i * d + c];
            snorm[ns] = band_w ? orc_band_len(K + (size_t)i * d, d, band_w, band_layout) : sqrt(n2);
            seed_of[i] = i;
            ++ns;
        }
    int joined = 0;
    for (int j = P; j < T - r; ++j) {
        if (kind[j] != 0) continue;
        const float* kj = K + (size_t)j * d;
        double n2 = 0.0;
        for (int c = 0; c < d; ++c) n2 += (chan_w ? (double)chan_w[c] : 1.0) * (double)kj[c] * (double)kj[c];
        double nj = band_w ? orc_band_len(kj, d, band_w, band_layout) : sqrt(n2);
        double best = -INFINITY, second = -INFINITY;
        int best_u = -1;
        for (int u = 0; u < ns; ++u) {           /* seeds[] ascends, so '>' keeps the smallest row on ties */
            const float* ku = K + (size_t)seeds[u] * d;
            double dot = 0.0;
            for (int c = 0; c < d; ++c) dot += (chan_w ? (double)chan_w[c] : 1.0) * (double)kj[c] * (double)ku[c];
            double sm = (nj > 0.0 && snorm[u] > 0.0) ? dot / (nj * snorm[u]) : 0.0;
            if (band_w)
                sm = (nj > 0.0 && snorm[u] > 0.0) ? 1.0 - orc_band_dist(kj, ku, d, band_w, band_layout) / (nj + snorm[u])
                                                  : 0.0;
            if (sm > best) { second = best; best = sm; best_u = u; }
            else if (sm > second) second = sm;
        }
        if (sim) sim[j] = best;
        if (sim2) sim2[j] = (ns > 1) ? second : -2.0;
        if (best_u >= 0 && best >= tau) {
            kind[j] = 5;
            seed_of[j] = seeds[best_u];
            ++joined;
        } else {
            *lost_mass += orc_a(s, mass_in, eps, j);
        }
    }
    for (int u = 0; u < ns; ++u) {
        double mG = 0.0;
        for (int i = P; i < T - r; ++i)
            if (seed_of[i] == seeds[u]) mG += orc_a(s, mass_in, eps, i);
        for (int i = P; i < T - r; ++i)
            if (seed_of[i] == seeds[u]) weight[i] = orc_a(s, mass_in, eps, i) / mG;
    }
    free(seeds);
    free(snorm);
    return joined == 0 ? ORC_MERGE_INACTIVE : 0;
}

/*
 * Compaction (Sec. 2.3: |R| <= B).  Output slots are the rows of kind 1..4 in
 * ascending row order; a representative sits at its seed's row.  A slot of
 * kind 4 holds k~ = sum_i w_i k_i, v~ = sum_i w_i v_i over its group (Sec. 2.4);
 * every other slot is a copy of its row.  slot_mass = sum of a_i over the
 * slot's members.  assign[i] = slot of row i's anchor or -1; weight of kept
 * singletons is set to 1 and of dropped rows to 0.
 */
void cask_oracle_compact(const float* K, const float* V, int T, int d, const uint8_t* kind,
                         const int* seed_of, double* weight, const double* s, double eps,
                         const double* mass_in, double* k_out, double* v_out, int* n_out, int* slot_src, uint8_t* slot_kind,
                         double* slot_mass, int* assign) {
    int n = 0;
    for (int i = 0; i < T; ++i) {
        assign[i] = -1;
        if (kind[i] >= 1 && kind[i] <= 4) {
            slot_src[n] = i;
            slot_kind[n] = kind[i];
            assign[i] = n;
            ++n;
        }
    }
    *n_out = n;
    for (int i = 0; i < T; ++i) {
        if (kind[i] == 5) assign[i] = assign[seed_of[i]];
        if (kind[i] >= 1 && kind[i] <= 3) weight[i] = 1.0;
        if (kind[i] == 0) weight[i] = 0.0;
    }
    for (int t = 0; t < n; ++t) {
        int src = slot_src[t];
        double* ko = k_out + (size_t)t * d;
        double* vo = v_out + (size_t)t * d;
        if (slot_kind[t] != 4) {
            for (int c = 0; c < d; ++c) { ko[c] = K[(size_t)src * d + c]; vo[c] = V[(size_t)src * d + c]; }
            slot_mass[t] = orc_a(s, mass_in, eps, src);
        } else {
            double mass = 0.0;
            for (int c = 0; c < d; ++c) { ko[c] = 0.0; vo[c] = 0.0; }
            for (int i = 0; i < T; ++i) {
                if (seed_of[i] != src || (kind[i] != 4 && kind[i] != 5)) continue;
                mass += orc_a(s, mass_in, eps, i);
                for (int c = 0; c < d; ++c) {
                    ko[c] += weight[i] * (double)K[(size_t)i * d + c];
                    vo[c] += weight[i] * (double)V[(size_t)i * d + c];
                }
            }
            slot_mass[t] = mass;
        }
    }
}

/*
 * Representative-set mass diagnostics (Sec. 2.6):
 *     rho_core = sum_{k in C} s_k / sum_{k in TopK} s_k,   rho_rep = sum_{k in R} s_k / sum_{k in TopK} s_k.
 * Reading: s is the score of this event; TopK is the B greatest rows of the whole cache (the best any
 * B-row cache could hold); C = recent + core rows; the mass of R is the mass its slots carry
 * (slot_mass: a kept row its a_i, a representative its group mass m_G).
 */
void cask_oracle_diagnostics(const double* s, int T, int B, const uint8_t* kind, const double* slot_mass,
                             int n_out, double* rho_core, double* rho_rep) {
    orc_item* it = (orc_item*)malloc(sizeof(orc_item) * (size_t)(T > 0 ? T : 1));
    for (int i = 0; i < T; ++i) { it[i].s = s[i]; it[i].i = i; }
    qsort(it, (size_t)T, sizeof(orc_item), orc_cmp);
    double top = 0.0, core = 0.0, rep = 0.0;
    for (int t = 0; t < T && t < B; ++t) top += it[t].s;
    for (int i = 0; i < T; ++i)
        if (kind[i] == 2 || kind[i] == 3) core += s[i];
    for (int t = 0; t < n_out; ++t) rep += slot_mass[t];
    *rho_core = top > 0.0 ? core / top : 0.0;
    *rho_rep = top > 0.0 ? rep / top : 0.0;
    free(it);
}

/*
 * Within-group dispersion, the first term of the perturbation bound of Sec. 2.6:
 *     sum over groups G of  sum_{i in G} a_i || k_i - k~_G ||_kappa ,
 * a_i the merge weights' numerators (orc_a), k~_G the representative as the cache holds it: k_rep[slot] is passed in,
 * rounded to the cache's number format by the caller (a lone seed is its own copy and adds nothing).  The norm is the
 * one of the merge geometry in use: Euclidean; sqrt(sum_c w_c x_c^2) with channel weights; sum_f w_f ||x_f||_2 with
 * band weights (reading: the paper names the norm ||.||_kappa and gives it no formula beyond d_kappa of Sec. 2.5).
 */
double cask_oracle_dispersion(const float* K, const double* s, int T, int d, double eps, const double* mass_in,
                              const uint8_t* kind, const int* assign, const float* k_rep, const float* chan_w,
                              const float* band_w, int band_layout) {
    double total = 0.0;
    double* dd = (double*)malloc(sizeof(double) * (size_t)d);
    for (int i = 0; i < T; ++i) {
        if (kind[i] != 4 && kind[i] != 5) continue;
        int slot = assign[i];
        if (slot < 0) continue;
        for (int c = 0; c < d; ++c) dd[c] = (double)K[(size_t)i * d + c] - (double)k_rep[(size_t)slot * d + c];
        double norm = 0.0;
        if (band_w) {
            for (int f = 0; f < d / 2; ++f) {
                int c0, c1;
                orc_band(f, d, band_layout, &c0, &c1);
                norm += (double)band_w[f] * sqrt(dd[c0] * dd[c0] + dd[c1] * dd[c1]);
            }
        } else {
            for (int c = 0; c < d; ++c) norm += (chan_w ? (double)chan_w[c] : 1.0) * dd[c] * dd[c];
            norm = sqrt(norm);
        }
        total += orc_a(s, mass_in, eps, i) * norm;
    }
    free(dd);
    return total;
}

/* The whole event for one unit, the steps above in order.  plan[8] is written. */
void cask_oracle_event(const float* K, const float* V, const float* Q, int T, int P, int B, int reserve,
                       int d, int g, int W, int causal, double gamma, double tau, double eps,
                       const double* lse_in, const double* mass_in, const float* chan_w, const float* band_w,
                       int band_layout, double* s, int* plan, uint8_t* kind,
                       int* seed_of, double* weight, double* sim, double* sim2, double* k_out, double* v_out,
                       int* n_out, int* slot_src, uint8_t* slot_kind, double* slot_mass, int* assign,
                       int* status, double* lost_mass, double* rho /* nullable [2]: core, rep */) {
    cask_oracle_score(K, Q, T, d, g, W, causal, lse_in, s, NULL);
    cask_oracle_plan(T, P, B, reserve, W, gamma, plan);
    for (int i = 0; i < T; ++i) weight[i] = 0.0;
    cask_oracle_prefix_evict(s, P, plan, kind);
    cask_oracle_select_core(s, T, P, plan, kind);
    int fl = cask_oracle_consolidate(K, s, T, P, d, plan, tau, eps, mass_in, chan_w, band_w, band_layout, kind, seed_of,
                                     weight, sim, sim2, lost_mass);
    if (!(plan[PL_FLAGS] & ORC_DECODE_CONSOLIDATED)) fl = 0;
    cask_oracle_compact(K, V, T, d, kind, seed_of, weight, s, eps, mass_in, k_out, v_out, n_out, slot_src,
                        slot_kind, slot_mass, assign);
    *status = plan[PL_FLAGS] | fl;
    if (rho) cask_oracle_diagnostics(s, T, B, kind, slot_mass, *n_out, rho, rho + 1);
}

/*
 * Many independent units (Sec. 2.3 constrains one cache at a time; nothing
 * couples units), rows contiguous: unit u owns rows [tok_off[u], tok_off[u+1])
 * of K, V and of every per-row output, slots [u*Bmax, (u+1)*Bmax) of the slot
 * outputs, and Q[u].  OpenMP runs units in parallel when compiled with it.
 */
void cask_oracle_event_batch(int n_units, const float* K, const float* V, const float* Q,
                             const int64_t* tok_off, const int* P, const int* B, const int* reserve,
                             int d, int g, int W, int causal, double gamma, double tau, double eps,
                             const double* mass_in /* nullable [sum T] */, const float* chan_w /* nullable [d] */,
                             const float* band_w /* nullable [d/2] */, int band_layout, int Bmax, double* s, int* plan, uint8_t* kind, int* seed_of, double* weight,
                             double* sim, double* sim2, double* k_out, double* v_out, int* n_out,
                             int* slot_src, uint8_t* slot_kind, double* slot_mass, int* assign,
                             int* status, double* lost_mass, double* rho /* nullable [n_units, 2] */) {
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int u = 0; u < n_units; ++u) {
        size_t a = (size_t)tok_off[u];
        int T = (int)(tok_off[u + 1] - tok_off[u]);
        size_t so = (size_t)u * (size_t)Bmax;
        cask_oracle_event(K + a * d, V + a * d, Q + (size_t)u * g * W * d, T, P[u], B[u], reserve[u], d, g,
                          W, causal, gamma, tau, eps, NULL, mass_in ? mass_in + a : NULL, chan_w, band_w, band_layout, s + a, plan + (size_t)u * 8, kind + a,
                          seed_of + a, weight + a, sim ? sim + a : NULL, sim2 ? sim2 + a : NULL,
                          k_out + so * d, v_out + so * d, n_out + u, slot_src + so, slot_kind + so,
                          slot_mass + so, assign + a, status + u, lost_mass + u, rho ? rho + 2 * (size_t)u : NULL);
    }
}

/*
 * Query-statistics scorer of the Phase-1 archive (App. B): the horizon kernel
 *     kappa_{pi_h}(omega) = E_{delta ~ pi_h}[ e^{i omega delta} ] = sum_n pi_h[n] e^{i omega delta_n}
 * for a discrete horizon distribution pi_h on the offsets delta_n, and the horizon-averaged mean score
 *     S_h(k, Delta) = Re sum_f mu_{h,f} conj(k_f) kappa_{pi_h}(omega_f) e^{i omega_f Delta} ,
 * with band f of a vector read as the complex number x[c0] + i x[c1] (channel pairs as in orc_band).  Reading: the
 * score of cache row i is the mean of S_h over the g query heads of the KV head, at Delta_i = delta[i] when the
 * caller gives offsets, else T - 1 - i (distance to the newest row).  The score is real and may be negative.
 * mu [g, d/2, 2] (re, im), pi [g, n_delta], delta_grid [n_delta], omega [d/2].
 */
void cask_oracle_score_stats(const float* K, int T, int d, int g, const float* mu, const double* pi,
                             const double* delta_grid, int n_delta, const double* omega, int band_layout,
                             const double* delta, double* s) {
    int nb = d / 2;
    double* kr = (double*)malloc(sizeof(double) * (size_t)g * nb);      /* kappa_{h,f}: re */
    double* ki = (double*)malloc(sizeof(double) * (size_t)g * nb);      /*              im */
    for (int h = 0; h < g; ++h)
        for (int f = 0; f < nb; ++f) {
            double re = 0.0, im = 0.0;
            for (int n = 0; n < n_delta; ++n) {
                re += pi[(size_t)h * n_delta + n] * cos(omega[f] * delta_grid[n]);
                im += pi[(size_t)h * n_delta + n] * sin(omega[f] * delta_grid[n]);
            }
            kr[h * nb + f] = re;
            ki[h * nb + f] = im;
        }
    for (int i = 0; i < T; ++i) {
        double D = delta ? delta[i] : (double)(T - 1 - i);
        double tot = 0.0;
        for (int h = 0; h < g; ++h)
            for (int f = 0; f < nb; ++f) {
                int c0, c1;
                orc_band(f, d, band_layout, &c0, &c1);
                double mr = mu[((size_t)h * nb + f) * 2], mi = mu[((size_t)h * nb + f) * 2 + 1];
                double xr = K[(size_t)i * d + c0], xi = -(double)K[(size_t)i * d + c1];      /* conj(k_f) */
                double ar = mr * xr - mi * xi, ai = mr * xi + mi * xr;                        /* mu conj(k) */
                double br = ar * kr[h * nb + f] - ai * ki[h * nb + f];                       /* ... kappa  */
                double bi = ar * ki[h * nb + f] + ai * kr[h * nb + f];
                tot += br * cos(omega[f] * D) - bi * sin(omega[f] * D);                      /* Re(... e^{i omega D}) */
            }
        s[i] = tot / g;
    }
    free(kr);
    free(ki);
}

/* Scores only, many units (used where only the dominant step is timed or compared). */
void cask_oracle_score_batch(int n_units, const float* K, const float* Q, const int64_t* tok_off, int d,
                             int g, int W, int causal, double* s, double* lse_out) {
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1)
#endif
    for (int u = 0; u < n_units; ++u) {
        size_t a = (size_t)tok_off[u];
        int T = (int)(tok_off[u + 1] - tok_off[u]);
        cask_oracle_score(K + a * d, Q + (size_t)u * g * W * d, T, d, g, W, causal, NULL, s + a,
                          lse_out ? lse_out + (size_t)u * g * W : NULL);
    }
}

/* Round doubles to the nearest bfloat16 value (ties to even), returned as float. */
void cask_oracle_round_bf16(const double* x, size_t n, float* out) {
    for (size_t i = 0; i < n; ++i) {
        double v = x[i];
        if (v == 0.0 || !isfinite(v)) { out[i] = (float)v; continue; }
        int e;
        frexp(v, &e);                 /* |v| in [2^(e-1), 2^e) */
        int q = e - 8;                /* 8 significant bits */
        if (q < -133) q = -133;       /* bf16 subnormal quantum */
        out[i] = (float)ldexp(nearbyint(ldexp(v, -q)), q);
    }
}

int cask_oracle_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}

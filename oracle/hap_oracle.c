/*
 * CPU oracle of the HAPMoE planner hot path -- TEST INFRASTRUCTURE, not a product path.
 * See hap_oracle.h.  Plain loops, fp64 for the cost formulas (one IEEE operation per
 * operator, no contraction: build with -ffp-contract=off), exact int64 afterwards.
 */
#include "hap_oracle.h"
#include <math.h>
#include <string.h>
#include <stdlib.h>
#ifdef _OPENMP
#include <omp.h>
#endif

typedef unsigned __int128 u128;

/* ------------------------------------------------------------------------------------ *
 * Cluster helpers: device counts per type and the slowest uplink of a type.
 * ------------------------------------------------------------------------------------ */
static void type_counts(const orc_problem *pr, int64_t *m)
{
    for (int h = 0; h < pr->T; ++h) m[h] = 0;
    for (int n = 0; n < pr->n_nodes; ++n) m[pr->node_type[n]] += pr->node_size[pr->node_type[n]];
}

static double type_bw_inter(const orc_problem *pr, int h)
{
    double best = 0.0;
    int seen = 0;
    for (int n = 0; n < pr->n_nodes; ++n)
        if (pr->node_type[n] == h) {
            if (!seen || pr->node_bw_inter[n] < best) best = pr->node_bw_inter[n];
            seen = 1;
        }
    return best;
}

/* ------------------------------------------------------------------------------------ *
 * Multiset permutations in lexicographic order (types ascending).
 * ------------------------------------------------------------------------------------ */
static uint64_t sat_mul_div(uint64_t r, uint64_t mul, uint64_t div, uint64_t sat)
{
    if (r >= sat) return sat;
    u128 v = (u128)r * mul / div;   /* exact: callers keep r*mul divisible by div */
    return v >= sat ? sat : (uint64_t)v;
}

/* number of distinct sequences with cnt[h] copies of type h, saturated at `sat`:
 * the product over types of C(placed + cnt[h], cnt[h]), each binomial built one factor at a time */
uint64_t orc_multiset_count(const int32_t *cnt, int T, uint64_t sat)
{
    uint64_t r = 1;
    int placed = 0;
    for (int h = 0; h < T; ++h) {
        for (int i = 1; i <= cnt[h]; ++i)
            r = sat_mul_div(r, (uint64_t)(placed + i), (uint64_t)i, sat);   /* C(placed+i, i) from C(placed+i-1, i-1) */
        placed += cnt[h];
    }
    return r;
}

int orc_unrank_multiset(const int32_t *cnt_in, int T, int PP, uint64_t idx, uint8_t *seq)
{
    int32_t cnt[ORC_MAX_TYPES];
    for (int h = 0; h < T; ++h) cnt[h] = cnt_in[h];
    for (int pos = 0; pos < PP; ++pos) {
        int chosen = -1;
        for (int h = 0; h < T && chosen < 0; ++h) {
            if (cnt[h] == 0) continue;
            cnt[h]--;
            uint64_t below = orc_multiset_count(cnt, T, UINT64_MAX);
            if (idx < below) chosen = h;
            else { idx -= below; cnt[h]++; }
        }
        if (chosen < 0) return -1;
        seq[pos] = (uint8_t)chosen;
    }
    return 0;
}

uint64_t orc_rank_multiset(const int32_t *cnt_in, int T, int PP, const uint8_t *seq)
{
    int32_t cnt[ORC_MAX_TYPES];
    uint64_t rank = 0;
    for (int h = 0; h < T; ++h) cnt[h] = cnt_in[h];
    for (int pos = 0; pos < PP; ++pos) {
        for (int h = 0; h < seq[pos]; ++h) {
            if (cnt[h] == 0) continue;
            cnt[h]--;
            rank += orc_multiset_count(cnt, T, UINT64_MAX);
            cnt[h]++;
        }
        cnt[seq[pos]]--;
    }
    return rank;
}

static uint64_t factorial_u64(int n)
{
    uint64_t r = 1;
    for (int i = 2; i <= n; ++i) r *= (uint64_t)i;
    return r;
}

/* ------------------------------------------------------------------------------------ *
 * Enumeration of the 6-D parallel space x micro-batch (order defines candidate indices).
 * ------------------------------------------------------------------------------------ */
int orc_enumerate(const orc_problem *pr, orc_pconf *out, uint64_t cap, uint64_t *n_pconf, uint64_t *n_cand)
{
    int64_t m[ORC_MAX_TYPES];
    type_counts(pr, m);
    int64_t W = 0;
    for (int h = 0; h < pr->T; ++h) W += m[h];
    uint64_t np = 0, off = 0;
    for (int ipp = 0; ipp < pr->npp; ++ipp) {
        int PP = pr->pp_list[ipp];
        if (PP > pr->N || PP > ORC_MAX_PP || W % PP != 0) continue;
        int64_t G = W / PP;
        /* mapping mode and count depend on (PP) only */
        int homog = 1;
        int32_t cnt[ORC_MAX_TYPES];
        for (int h = 0; h < pr->T; ++h) {
            if (m[h] % G != 0) homog = 0;
            cnt[h] = (int32_t)(m[h] / G);
        }
        uint64_t nms = homog ? orc_multiset_count(cnt, pr->T, UINT64_MAX) : 0;
        int mode = (homog && nms <= pr->map_cap) ? ORC_MODE_MULTISET : ORC_MODE_BLOCK;
        uint64_t nmap = mode == ORC_MODE_MULTISET ? nms : factorial_u64(pr->T);
        for (int itp = 0; itp < pr->ntp; ++itp) {
            int TP = pr->tp_list[itp];
            if (G % TP != 0 || TP > pr->tp_max || pr->nq % TP != 0 || pr->nkv % TP != 0) continue;
            for (int icp = 0; icp < pr->ncp; ++icp) {
                int CP = pr->cp_list[icp];
                if (G % ((int64_t)TP * CP) != 0 || pr->S % (2 * CP) != 0) continue;
                int64_t DP = G / ((int64_t)TP * CP);
                for (int iep = 0; iep < pr->nep; ++iep) {
                    int EP = pr->ep_list[iep];
                    if (pr->E % EP != 0 || G % EP != 0) continue;
                    for (int itpe = 0; itpe < pr->ntpe; ++itpe) {
                        int TPE = pr->tpe_list[itpe];
                        if (G % ((int64_t)EP * TPE) != 0 || TPE > pr->tp_max) continue;
                        int64_t EDP = G / ((int64_t)EP * TPE);
                        for (int ib = 0; ib < pr->nmb; ++ib) {
                            int b = pr->mb_list[ib];
                            if (pr->GB % (DP * b) != 0) continue;
                            int64_t M = pr->GB / (DP * b);
                            if (out) {
                                if (np >= cap) return -2;
                                orc_pconf *q = &out[np];
                                q->PP = PP; q->TP = TP; q->CP = CP; q->DP = (int32_t)DP; q->EP = EP;
                                q->TPE = TPE; q->b = b; q->M = (int32_t)M; q->EDP = (int32_t)EDP;
                                q->G = (int32_t)G; q->itp = itp; q->icp = icp; q->ib = ib; q->iep = iep;
                                q->mode = mode; q->pad = 0; q->nmap = nmap; q->offset = off;
                            }
                            off += nmap * (uint64_t)pr->n_rc;
                            np++;
                        }
                    }
                }
            }
        }
    }
    *n_pconf = np;
    *n_cand = off;
    return 0;
}

/* ------------------------------------------------------------------------------------ *
 * Mapping of device groups to stages.
 * ------------------------------------------------------------------------------------ */
int orc_decode(const orc_problem *pr, const orc_pconf *pc, uint64_t map_idx, orc_mapping *out)
{
    int64_t m[ORC_MAX_TYPES];
    type_counts(pr, m);
    const int PP = pc->PP, T = pr->T;
    const int64_t G = pc->G;
    if (map_idx >= pc->nmap) return -1;
    memset(out, 0, sizeof(*out));
    out->PP = PP;
    /* per stage: type and position (within that type's device line) of first and last device */
    int tfirst[ORC_MAX_PP], tlast[ORC_MAX_PP];
    int64_t ofirst[ORC_MAX_PP], olast[ORC_MAX_PP];
    if (pc->mode == ORC_MODE_MULTISET) {
        int32_t cnt[ORC_MAX_TYPES];
        uint8_t seq[ORC_MAX_PP];
        int used[ORC_MAX_TYPES] = {0, 0, 0, 0};
        for (int h = 0; h < T; ++h) cnt[h] = (int32_t)(m[h] / G);
        if (orc_unrank_multiset(cnt, T, PP, map_idx, seq) != 0) return -1;
        for (int s = 0; s < PP; ++s) {
            int h = seq[s];
            int q = used[h]++;
            out->mask[s] = (uint8_t)(1u << h);
            tfirst[s] = tlast[s] = h;
            ofirst[s] = (int64_t)q * G;
            olast[s] = (int64_t)(q + 1) * G - 1;
        }
    } else {
        /* map_idx-th permutation of the types in lexicographic order */
        int sigma[ORC_MAX_TYPES], avail[ORC_MAX_TYPES];
        uint64_t idx = map_idx;
        for (int h = 0; h < T; ++h) avail[h] = h;
        for (int pos = 0; pos < T; ++pos) {
            uint64_t f = factorial_u64(T - 1 - pos);
            int pick = (int)(idx / f);
            idx %= f;
            sigma[pos] = avail[pick];
            for (int t = pick; t + 1 < T - pos; ++t) avail[t] = avail[t + 1];
        }
        int64_t start[ORC_MAX_TYPES + 1];
        start[0] = 0;
        for (int bq = 0; bq < T; ++bq) start[bq + 1] = start[bq] + m[sigma[bq]];
        for (int s = 0; s < PP; ++s) {
            int64_t lo = (int64_t)s * G, hi = (int64_t)(s + 1) * G - 1;
            for (int bq = 0; bq < T; ++bq) {
                if (start[bq + 1] <= lo || start[bq] > hi) continue;   /* block does not overlap */
                out->mask[s] |= (uint8_t)(1u << sigma[bq]);
                if (start[bq] <= lo && lo < start[bq + 1]) { tfirst[s] = sigma[bq]; ofirst[s] = lo - start[bq]; }
                if (start[bq] <= hi && hi < start[bq + 1]) { tlast[s] = sigma[bq]; olast[s] = hi - start[bq]; }
            }
        }
    }
    for (int s = 1; s < PP; ++s) {
        int ta = tlast[s - 1], tb = tfirst[s];
        out->ha[s] = (uint8_t)ta;
        out->hb[s] = (uint8_t)tb;
        if (ta != tb) out->cls[s] = ORC_CROSS;
        else out->cls[s] = (olast[s - 1] / pr->node_size[ta] == ofirst[s] / pr->node_size[tb]) ? ORC_INTRA : ORC_INTER;
    }
    return 0;
}

/* ------------------------------------------------------------------------------------ *
 * Layer cost (Eq. 2, Eq. 3, imbalance scaling) and stage-level coefficients.
 * c2 / c2f: [T][N][2] (forward, backward); coef / coeff: [T][ORC_NCOEF].
 * ------------------------------------------------------------------------------------ */
typedef struct { const orc_problem *pr; int h; double bw_inter; } linkctx;

static int link_cls(const linkctx *lc, int64_t ext) { return ext <= lc->pr->node_size[lc->h] ? ORC_INTRA : ORC_INTER; }
static double link_bw(const linkctx *lc, int cls) { return cls == ORC_INTRA ? lc->pr->bw_intra[lc->h] : lc->bw_inter; }

/* Volume term of a communication primitive (the communication-primitive table of Sec. 3.4): the time to move
 * `vol` bytes over a link of class c with nominal bandwidth bw is vol / bw divided by the link's profiled
 * efficiency at that message size, piecewise linear between the profiled sizes and constant outside them.
 * Without a table the efficiency is 1 and the term is vol / bw. */
static double link_eff(const orc_problem *pr, int c, double vol)
{
    const int n = pr->n_fsize;
    const double *sz = pr->fsize, *e = pr->feff + (size_t)c * n;
    if (vol <= sz[0]) return e[0];
    if (vol >= sz[n - 1]) return e[n - 1];
    int i = 0;
    while (vol >= sz[i + 1]) ++i;
    return e[i] + (vol - sz[i]) * ((e[i + 1] - e[i]) / (sz[i + 1] - sz[i]));
}

static double xfer(const orc_problem *pr, int c, double vol, double bw)
{
    const double t = vol / bw;
    if (pr->n_fsize <= 0) return t;
    return t / link_eff(pr, c, vol);
}

/* ring-style collective over w ranks spanning `ext` devices moving D bytes */
static double coll(const linkctx *lc, int64_t w, int64_t ext, double D)
{
    if (w == 1) return 0.0;
    int c = link_cls(lc, ext);
    double lat = lc->pr->alpha[c] * (double)(w - 1);
    double vol = (D * (double)(w - 1)) / (double)w;
    return lat + xfer(lc->pr, c, vol, link_bw(lc, c));
}

int orc_layer_costs(const orc_problem *pr, const orc_pconf *pc, int64_t *c2, double *c2f,
                    int64_t *coef, double *coeff)
{
    const int N = pr->N, T = pr->T;
    const int TP = pc->TP, CP = pc->CP, DP = pc->DP, EP = pc->EP, TPE = pc->TPE, EDP = pc->EDP, b = pc->b;
    const int64_t G = pc->G;
    const int64_t tok = (int64_t)b * pr->S / CP;
    const int64_t Hkv = (int64_t)pr->H * pr->nkv / pr->nq;
    const int64_t H = pr->H;
    double bwi[ORC_MAX_TYPES];
    for (int h = 0; h < T; ++h) bwi[h] = type_bw_inter(pr, h);

    for (int h = 0; h < T; ++h) {
        linkctx lc = { pr, h, bwi[h] };
        const double thb = (double)tok * (double)H;        /* token*hidden elements per rank */
        const double Dtp = thb * pr->beta;
        const double imb = 1.0 + pr->gamma * (pr->rho[pc->iep] - 1.0);
        /* expert dispatch / combine: Eq. 3 bytes, best of all-to-all and all-gather */
        double tdisp;
        if (EP == 1) tdisp = 0.0;
        else {
            double Dmoe = ((thb * pr->beta) * (double)pr->k) * (1.0 - 1.0 / (double)EP);
            double Dag = (thb * pr->beta) * (double)(EP - 1);
            int c = link_cls(&lc, (int64_t)EP * TPE);
            double fa = pr->alpha[c] * (double)(EP - 1) + xfer(pr, c, Dmoe, link_bw(&lc, c));
            double fg = pr->alpha[c] * (double)(EP - 1) + xfer(pr, c, Dag, link_bw(&lc, c));
            tdisp = (fa <= fg) ? fa : fg;
        }
        const double ttpA = 2.0 * coll(&lc, TP, TP, Dtp);
        const double ttpD = 2.0 * coll(&lc, TP, TP, Dtp);
        const double ttpM = 2.0 * coll(&lc, TPE, TPE, Dtp);
        const double Dkv = ((((2.0 * (double)b) * (double)pr->S) * (double)Hkv) * pr->beta) / (double)TP;
        const double tcp = coll(&lc, CP, (int64_t)TP * CP, Dkv);
        const double tr = pr->croute[h] * thb;
        double commF[2], commB[2];
        commF[ORC_DENSE] = pr->ovl_tp * (ttpA + ttpD) + pr->ovl_cp * tcp;
        commB[ORC_DENSE] = pr->ovl_tp * (ttpA + ttpD) + pr->ovl_cp * (2.0 * tcp);
        commF[ORC_MOE] = pr->ovl_tp * (ttpA + ttpM) + pr->ovl_cp * tcp;
        commB[ORC_MOE] = pr->ovl_tp * (ttpA + ttpM) + pr->ovl_cp * (2.0 * tcp);

        const int64_t i4 = (((int64_t)h * pr->ntp + pc->itp) * pr->ncp + pc->icp) * pr->nmb + pc->ib;
        for (int l = 0; l < N; ++l) {
            const double a = pr->tdf[i4 * N + l], f = pr->tff[i4 * N + l];
            const double ab = pr->tdb[i4 * N + l], fb = pr->tfb[i4 * N + l];
            double cf, cb;
            if (pr->kind[l] == ORC_DENSE) {
                cf = a + commF[ORC_DENSE];
                cb = ab + commB[ORC_DENSE];
            } else {
                const double den = (pr->eta[h] * (double)EP) * (double)TPE;
                const double xf = (pr->kappa * f) / den;
                const double mf = (xf + 2.0 * tdisp) * imb;
                cf = (((a - f) + mf) + tr) + commF[ORC_MOE];
                const double xb = (pr->kappa * fb) / den;
                const double mb = (xb + 2.0 * tdisp) * imb;
                cb = (((ab - fb) + mb) + 2.0 * tr) + commB[ORC_MOE];
            }
            if (c2f) { c2f[((int64_t)h * N + l) * 2] = cf; c2f[((int64_t)h * N + l) * 2 + 1] = cb; }
            if (c2) { c2[((int64_t)h * N + l) * 2] = llrint(cf); c2[((int64_t)h * N + l) * 2 + 1] = llrint(cb); }
        }

        /* stage-level coefficients */
        double v[ORC_NCOEF];
        v[ORC_KPRE] = pr->tpre[i4];
        v[ORC_KPOST] = pr->tpost[i4];
        v[ORC_KP2P_INTRA] = 2.0 * (pr->alpha[ORC_INTRA] + xfer(pr, ORC_INTRA, Dtp / (double)TP, pr->bw_intra[h]));
        v[ORC_KP2P_INTER] = 2.0 * (pr->alpha[ORC_INTER] + xfer(pr, ORC_INTER, Dtp / (double)TP, bwi[h]));
        for (int h2 = 0; h2 < ORC_MAX_TYPES; ++h2) {
            double bo = h2 < T ? bwi[h2] : bwi[h];
            double bmin = bwi[h] < bo ? bwi[h] : bo;
            v[ORC_KP2P_CROSS + h2] = 2.0 * (pr->alpha[ORC_CROSS] + xfer(pr, ORC_CROSS, Dtp / (double)TP, bmin * pr->chi));
        }
        const double shd = 6.0 + 12.0 / (double)((int64_t)DP * CP);
        const double she = 6.0 + 12.0 / (double)EDP;
        const int64_t Pattn = H * (H + 2 * Hkv) + H * H + 2 * H;
        const int64_t Pffn_d = 3 * H * (int64_t)pr->F_dense, Pffn_e = 3 * H * (int64_t)pr->F_exp;
        const int64_t Pe = (int64_t)(pr->E / EP) * Pffn_e;
        int64_t Pd[2];
        Pd[ORC_DENSE] = Pattn + Pffn_d;
        Pd[ORC_MOE] = Pattn + (int64_t)pr->n_shared * Pffn_e;
        const int64_t Prt = H * (int64_t)pr->E;
        v[ORC_MW + ORC_DENSE] = ((double)Pd[ORC_DENSE] / (double)TP) * shd;
        v[ORC_MW + ORC_MOE] = ((double)Pd[ORC_MOE] / (double)TP + (double)Prt) * shd + ((double)Pe / (double)TPE) * she;
        for (int kd = 0; kd < 2; ++kd) v[ORC_MA + kd] = (thb * pr->act_coef[kd]) / (double)TP;
        v[ORC_MX] = ((2.0 * ((thb * pr->beta) * (double)pr->k)) * (1.0 - 1.0 / (double)EP)) * pr->capf
                    + ((double)tok * (double)pr->E) * 4.0;
        v[ORC_MPRE] = (((double)pr->V * (double)H) / (double)TP) * shd;
        v[ORC_MPOST] = v[ORC_MPRE];
        const int cG = link_cls(&lc, G);
        const double bwG = link_bw(&lc, cG);
        const int64_t wd = (int64_t)DP * CP;
        const double vfd = (double)(wd - 1) / (double)wd, vfe = (double)(EDP - 1) / (double)EDP;
        for (int kd = 0; kd < 2; ++kd) {
            const int64_t Pdd = Pd[kd] + (kd == ORC_MOE ? Prt : 0);
            const double Pel = kd == ORC_MOE ? (double)Pe / (double)TPE : 0.0;
            v[ORC_SBW + kd] = pr->ovl_dp * (xfer(pr, cG, (6.0 * ((double)Pdd / (double)TP)) * vfd, bwG)
                                            + xfer(pr, cG, (6.0 * Pel) * vfe, bwG));
            v[ORC_OPT + kd] = pr->copt[h] * ((double)Pdd / (double)((int64_t)TP * DP * CP) + Pel / (double)EDP);
        }
        v[ORC_SLAT] = pr->ovl_dp * (pr->alpha[cG] * (2.0 * (double)(wd - 1) + 2.0 * (double)(EDP - 1)));
        /* dispatch and combine of one MoE layer, forward and backward (the 2 t_disp per direction of Eq. 2, with
         * its imbalance factor), when the expert-parallel group spans device types: Eq. 3's volumes over the
         * cross-type link class at chi times this type's inter-node bandwidth.  Used by Pruning 3 only. */
        if (EP == 1) v[ORC_KXD] = 0.0;
        else {
            double Dmoe = ((thb * pr->beta) * (double)pr->k) * (1.0 - 1.0 / (double)EP);
            double Dag = (thb * pr->beta) * (double)(EP - 1);
            double bx = bwi[h] * pr->chi;
            double fa = pr->alpha[ORC_CROSS] * (double)(EP - 1) + xfer(pr, ORC_CROSS, Dmoe, bx);
            double fg = pr->alpha[ORC_CROSS] * (double)(EP - 1) + xfer(pr, ORC_CROSS, Dag, bx);
            v[ORC_KXD] = (4.0 * ((fa <= fg) ? fa : fg)) * imb;
        }
        for (int q = 0; q < ORC_NCOEF; ++q) {
            if (coeff) coeff[h * ORC_NCOEF + q] = v[q];
            if (coef) coef[h * ORC_NCOEF + q] = llrint(v[q]);
        }
    }
    return 0;
}

/* ------------------------------------------------------------------------------------ *
 * Stage cost with minimal feasible recomputation (integer arithmetic).
 * Stage index i is 1-based; the span is layers a..b-1, i.e. (a, b] in prefix terms.
 * ------------------------------------------------------------------------------------ */
static int64_t mask_max(const orc_problem *pr, unsigned mask, const int64_t *coef, int q)
{
    int64_t best = 0;
    int seen = 0;
    for (int h = 0; h < pr->T; ++h)
        if (mask & (1u << h)) {
            int64_t x = coef[h * ORC_NCOEF + q];
            if (!seen || x > best) best = x;
            seen = 1;
        }
    return best;
}

int orc_window(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, int32_t *nmin, int32_t *nmax)
{
    const int PP = pc->PP, N = pr->N;
    if (pr->uniform) {
        /* ablation "non-uniform partitioning disabled": every stage takes floor(N/PP) or ceil(N/PP) layers */
        for (int s = 0; s < PP; ++s) { nmin[s] = N / PP; nmax[s] = (N + PP - 1) / PP; }
        return 2;
    }
    if (pr->delta_q < 0) {
        for (int s = 0; s < PP; ++s) { nmin[s] = 1; nmax[s] = N - PP + 1; }
        return 0;
    }
    int64_t Pst[ORC_MAX_PP], Ps = 0;
    for (int s = 0; s < PP; ++s) {
        int64_t p = 0;
        int seen = 0;
        for (int h = 0; h < pr->T; ++h)
            if (mp->mask[s] & (1u << h)) {
                if (!seen || pr->P[h] < p) p = pr->P[h];
                seen = 1;
            }
        Pst[s] = p;
        Ps += p;
    }
    for (int s = 0; s < PP; ++s) {
        int64_t lo = ((int64_t)(1024 - pr->delta_q) * Pst[s] * N) / (1024 * Ps);
        int64_t num = (int64_t)(1024 + pr->delta_q) * Pst[s] * N, den = 1024 * Ps;
        int64_t hi = (num + den - 1) / den;
        if (lo < 1) lo = 1;
        if (hi > N - PP + 1) hi = N - PP + 1;
        nmin[s] = (int32_t)lo;
        nmax[s] = (int32_t)hi;
    }
    return 1;
}

/* Per-candidate stage data: the rows of Sec. "stage cost" built once, then every span is O(R). */
typedef struct {
    int N, PP, R;
    int64_t M;
    uint32_t rc_mask;
    const int32_t *xi_q, *tau_q;
    int64_t PF[ORC_MAX_PP][ORC_MAX_N + 1];   /* prefix sums of the forward row of stage s */
    int64_t PB[ORC_MAX_PP][ORC_MAX_N + 1];   /* prefix sums of the backward row of stage s */
    int64_t PW[ORC_MAX_N + 1], PA[ORC_MAX_N + 1];   /* weight / activation bytes (type independent) */
    int32_t PK[ORC_MAX_N + 1];               /* number of MoE layers among the first l */
    int64_t cap[ORC_MAX_PP], K[ORC_MAX_PP], mpre, mpost, mx;
    int32_t nmin[ORC_MAX_PP], nmax[ORC_MAX_PP];
} stage_ctx;

static void ctx_build(stage_ctx *cx, const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                      uint32_t rc_mask, const int64_t *c2, const int64_t *coef)
{
    const int N = pr->N, PP = pc->PP;
    cx->N = N; cx->PP = PP; cx->R = pr->R; cx->M = pc->M; cx->rc_mask = rc_mask;
    cx->xi_q = pr->xi_q; cx->tau_q = pr->tau_q;
    orc_window(pr, pc, mp, cx->nmin, cx->nmax);
    cx->PW[0] = cx->PA[0] = 0; cx->PK[0] = 0;
    for (int l = 0; l < N; ++l) {
        /* weight / activation bytes do not depend on the device type: row of type 0 */
        cx->PW[l + 1] = cx->PW[l] + coef[ORC_MW + pr->kind[l]];
        cx->PA[l + 1] = cx->PA[l] + coef[ORC_MA + pr->kind[l]];
        cx->PK[l + 1] = cx->PK[l] + (pr->kind[l] == ORC_MOE ? 1 : 0);
    }
    cx->mpre = coef[ORC_MPRE]; cx->mpost = coef[ORC_MPOST]; cx->mx = coef[ORC_MX];
    for (int s = 0; s < PP; ++s) {
        const unsigned mask = mp->mask[s];
        const int i = s + 1;
        /* a (possibly mixed) stage runs each layer at the pace of its slowest member type */
        cx->PF[s][0] = cx->PB[s][0] = 0;
        for (int l = 0; l < N; ++l) {
            int64_t F = 0, Bk = 0;
            int seen = 0;
            for (int h = 0; h < pr->T; ++h)
                if (mask & (1u << h)) {
                    int64_t qf = c2[((int64_t)h * N + l) * 2], qb = c2[((int64_t)h * N + l) * 2 + 1];
                    if (!seen || qf > F) F = qf;
                    if (!seen || qb > Bk) Bk = qb;
                    seen = 1;
                }
            cx->PF[s][l + 1] = cx->PF[s][l] + F;
            cx->PB[s][l + 1] = cx->PB[s][l] + Bk;
        }
        /* it must fit its smallest member */
        int64_t cap = 0;
        int seen = 0;
        for (int h = 0; h < pr->T; ++h)
            if (mask & (1u << h)) {
                if (!seen || pr->cap_eff[h] < cap) cap = pr->cap_eff[h];
                seen = 1;
            }
        cx->cap[s] = cap;
        /* stage constant: embedding / head work and the p2p transfer into this stage */
        int64_t K = 0;
        if (i == 1) K += mask_max(pr, mask, coef, ORC_KPRE);
        if (i == PP) K += mask_max(pr, mask, coef, ORC_KPOST);
        if (i > 1) {
            int hb = mp->hb[s], ha = mp->ha[s];
            if (mp->cls[s] == ORC_INTRA) K += coef[hb * ORC_NCOEF + ORC_KP2P_INTRA];
            else if (mp->cls[s] == ORC_INTER) K += coef[hb * ORC_NCOEF + ORC_KP2P_INTER];
            else K += coef[hb * ORC_NCOEF + ORC_KP2P_CROSS + ha];
        }
        cx->K[s] = K;
    }
}

/* cost of stage i (1-based) holding layers a..b-1 */
static int64_t ctx_stage_cost(const stage_ctx *cx, int i, int a, int b, int *r_out)
{
    const int s = i - 1, PP = cx->PP;
    if (r_out) *r_out = -1;
    const int n = b - a;
    if (n < cx->nmin[s] || n > cx->nmax[s]) return ORC_INF;          /* Pruning 1: load-balance window */
    /* memory: M_w + M_act + M_moe-extra */
    const int has_moe = cx->PK[b] - cx->PK[a] > 0;
    const int64_t Wb = (cx->PW[b] - cx->PW[a]) + (i == 1 ? cx->mpre : 0) + (i == PP ? cx->mpost : 0)
                       + (has_moe ? cx->mx : 0);
    const int64_t Mstore = cx->M < PP - i + 1 ? cx->M : PP - i + 1;    /* 1F1B in-flight micro-batches */
    const int64_t A = Mstore * (cx->PA[b] - cx->PA[a]);
    int rstar = -1;
    for (int r = 0; r < cx->R && rstar < 0; ++r)
        if ((cx->rc_mask >> r) & 1u)
            if (Wb + ((int64_t)cx->xi_q[r] * A) / 1024 <= cx->cap[s]) rstar = r;    /* minimal feasible level */
    if (rstar < 0) return ORC_INF;                                   /* Pruning 2: memory */
    if (r_out) *r_out = rstar;
    const int64_t SF = cx->PF[s][b] - cx->PF[s][a], SB = cx->PB[s][b] - cx->PB[s][a];
    return SF + SB + ((int64_t)cx->tau_q[rstar] * SF) / 1024 + cx->K[s];
}

int64_t orc_stage_cost(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                       uint32_t rc_mask, const int64_t *c2, const int64_t *coef,
                       int i, int a, int b, int *r_out)
{
    stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
    if (!cx) return -1;
    ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
    int64_t c = ctx_stage_cost(cx, i, a, b, r_out);
    free(cx);
    return c;
}


/* Pruning 3 (heterogeneous communication): the candidate is dropped when its cross-type communication time
 * per micro-batch exceeds eta times the mean stage time, T_hetero > eta * (1/PP) * sum_i c_i.
 * T_hetero is the stage-to-stage transfers over cross-type links; with het_coll set it also holds, for every
 * stage whose devices are of more than one type (its expert-parallel groups leave a homogeneous sub-cluster,
 * the case Sec. 3.5 names), the dispatch and combine traffic of the stage's MoE layers re-timed on the
 * cross-type link: n_moe(stage) times the slowest member type's coefficient ORC_KXD.  The stage times
 * themselves are not changed by the option.
 * eta is given in 1/1024 (eta_q = 2048 is the paper's default eta = 2); eta_q <= 0 switches the rule off.
 * n[s] = layers of stage s of the chosen partition. */
static int64_t hetero_comm(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, const int64_t *coef,
                           const uint8_t *n)
{
    int64_t t = 0;
    for (int s = 1; s < pc->PP; ++s)
        if (mp->cls[s] == ORC_CROSS) t += coef[mp->hb[s] * ORC_NCOEF + ORC_KP2P_CROSS + mp->ha[s]];
    if (pr->het_coll) {
        int a = 0;
        for (int s = 0; s < pc->PP; ++s) {
            const unsigned mask = mp->mask[s];
            if (mask & (mask - 1)) {                       /* more than one device type in the stage */
                int64_t n_moe = 0;
                for (int l = a; l < a + n[s]; ++l) n_moe += pr->kind[l] == ORC_MOE;
                t += n_moe * mask_max(pr, mask, coef, ORC_KXD);
            }
            a += n[s];
        }
    }
    return t;
}

static int pruned_by_hetero_comm(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                                 const int64_t *coef, int64_t sum_stage, const uint8_t *n)
{
    if (pr->eta_q <= 0) return 0;
    return hetero_comm(pr, pc, mp, coef, n) * (int64_t)pc->PP * 1024 > (int64_t)pr->eta_q * sum_stage;
}

/* ------------------------------------------------------------------------------------ *
 * Min-max pipeline partitioning recurrence, backtrace and Eq. 4 closed form.
 * dp_table: [(PP+1)][(N+1)] or NULL; ch_table: same shape, 255 where undefined.
 * ------------------------------------------------------------------------------------ */
int orc_candidate(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                  const int64_t *c2, const int64_t *coef, orc_result *res,
                  int64_t *dp_table, uint8_t *ch_table)
{
    const int N = pr->N, PP = pc->PP;
    stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
    int64_t *DPt = (int64_t *)malloc(sizeof(int64_t) * (size_t)(PP + 1) * (N + 1));
    uint8_t *CH = (uint8_t *)malloc((size_t)(PP + 1) * (N + 1));
    if (!DPt || !CH || !cx) { free(DPt); free(CH); free(cx); return -1; }
    ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
#define DPAT(i, j) DPt[(size_t)(i) * (N + 1) + (j)]
#define CHAT(i, j) CH[(size_t)(i) * (N + 1) + (j)]
    for (int i = 0; i <= PP; ++i)
        for (int j = 0; j <= N; ++j) { DPAT(i, j) = ORC_INF; CHAT(i, j) = 255; }
    DPAT(0, 0) = 0;
    for (int i = 1; i <= PP; ++i)
        for (int j = i; j <= N - PP + i; ++j)
            for (int k = i - 1; k <= j - 1; ++k) {
                if (DPAT(i - 1, k) >= ORC_INF) continue;
                int64_t c = ctx_stage_cost(cx, i, k, j, NULL);
                int64_t v = DPAT(i - 1, k) > c ? DPAT(i - 1, k) : c;
                if (v < DPAT(i, j)) { DPAT(i, j) = v; CHAT(i, j) = (uint8_t)k; }   /* strict: smallest k wins */
            }
    memset(res, 0, sizeof(*res));
    res->bottleneck = DPAT(PP, N);
    if (dp_table) memcpy(dp_table, DPt, sizeof(int64_t) * (size_t)(PP + 1) * (N + 1));
    if (ch_table) memcpy(ch_table, CH, (size_t)(PP + 1) * (N + 1));
    if (res->bottleneck >= ORC_INF) {
        res->T_iter = res->T_pipe = ORC_INF;
        free(DPt); free(CH); free(cx);
        return 1;
    }
    /* backtrace */
    int64_t sum = 0, mx = 0, tsync = 0, topt = 0;
    int j = N;
    for (int i = PP; i >= 1; --i) {
        int k = CHAT(i, j), r;
        int64_t c = ctx_stage_cost(cx, i, k, j, &r);
        res->n[i - 1] = (uint8_t)(j - k);
        res->r[i - 1] = (uint8_t)r;
        res->c[i - 1] = c;
        sum += c;
        if (c > mx) mx = c;
        /* gradient synchronisation and optimizer step of this stage (after the partition is fixed) */
        unsigned mask = mp->mask[i - 1];
        int64_t sy = mask_max(pr, mask, coef, ORC_SLAT), op = 0;
        for (int l = k; l < j; ++l) {
            sy += mask_max(pr, mask, coef, ORC_SBW + pr->kind[l]);
            op += mask_max(pr, mask, coef, ORC_OPT + pr->kind[l]);
        }
        if (sy > tsync) tsync = sy;
        if (op > topt) topt = op;
        j = k;
    }
    res->T_pipe = sum + (int64_t)(pc->M - 1) * mx;     /* sum(stage) + (M-1) * max(stage) */
    res->T_sync = tsync;
    res->T_opt = topt;
    res->T_iter = res->T_pipe + tsync + topt;
    if (pruned_by_hetero_comm(pr, pc, mp, coef, sum, res->n)) res->T_iter = res->T_pipe = ORC_INF;   /* Pruning 3 */
    free(DPt); free(CH); free(cx);
#undef DPAT
#undef CHAT
    return 0;
}

/* ------------------------------------------------------------------------------------ *
 * Refinement (lexicographic optimum): among the partitions whose largest stage cost equals the
 * bottleneck B* of the min-max recurrence, take the one with the smallest SUM of stage costs
 * (Eq. 4's T_edge term), smallest split on ties.  This removes the dependence of the iteration
 * time on which of the bottleneck-optimal partitions the min-max tie-break happened to pick.
 * ------------------------------------------------------------------------------------ */
int orc_candidate_refined(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                          const int64_t *c2, const int64_t *coef, orc_result *res)
{
    const int N = pr->N, PP = pc->PP;
    orc_result first;
    int rc0 = orc_candidate(pr, pc, mp, rc_mask, c2, coef, &first, NULL, NULL);
    if (rc0 != 0) { *res = first; return rc0; }          /* infeasible (or error): nothing to refine */
    const int64_t Bstar = first.bottleneck;
    stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
    int64_t *D = (int64_t *)malloc(sizeof(int64_t) * (size_t)(PP + 1) * (N + 1));
    uint8_t *CH = (uint8_t *)malloc((size_t)(PP + 1) * (N + 1));
    if (!D || !CH || !cx) { free(D); free(CH); free(cx); return -1; }
    ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
#define DAT(i, j) D[(size_t)(i) * (N + 1) + (j)]
#define CHAT(i, j) CH[(size_t)(i) * (N + 1) + (j)]
    for (int i = 0; i <= PP; ++i)
        for (int j = 0; j <= N; ++j) { DAT(i, j) = ORC_INF; CHAT(i, j) = 255; }
    DAT(0, 0) = 0;
    for (int i = 1; i <= PP; ++i)
        for (int j = i; j <= N - PP + i; ++j)
            for (int k = i - 1; k <= j - 1; ++k) {
                if (DAT(i - 1, k) >= ORC_INF) continue;
                int64_t c = ctx_stage_cost(cx, i, k, j, NULL);
                if (c > Bstar) continue;                         /* keep the bottleneck optimal */
                int64_t v = DAT(i - 1, k) + c;
                if (v < DAT(i, j)) { DAT(i, j) = v; CHAT(i, j) = (uint8_t)k; }   /* strict: smallest k wins */
            }
    memset(res, 0, sizeof(*res));
    res->bottleneck = Bstar;
    int64_t sum = 0, mx = 0, tsync = 0, topt = 0;
    int j = N;
    for (int i = PP; i >= 1; --i) {
        int k = CHAT(i, j), r;
        int64_t c = ctx_stage_cost(cx, i, k, j, &r);
        res->n[i - 1] = (uint8_t)(j - k);
        res->r[i - 1] = (uint8_t)r;
        res->c[i - 1] = c;
        sum += c;
        if (c > mx) mx = c;
        unsigned mask = mp->mask[i - 1];
        int64_t sy = mask_max(pr, mask, coef, ORC_SLAT), op = 0;
        for (int l = k; l < j; ++l) {
            sy += mask_max(pr, mask, coef, ORC_SBW + pr->kind[l]);
            op += mask_max(pr, mask, coef, ORC_OPT + pr->kind[l]);
        }
        if (sy > tsync) tsync = sy;
        if (op > topt) topt = op;
        j = k;
    }
    res->T_pipe = sum + (int64_t)(pc->M - 1) * mx;
    res->T_sync = tsync;
    res->T_opt = topt;
    res->T_iter = res->T_pipe + tsync + topt;
    if (pruned_by_hetero_comm(pr, pc, mp, coef, sum, res->n)) res->T_iter = res->T_pipe = ORC_INF;   /* Pruning 3 */
    free(D); free(CH); free(cx);
#undef DAT
#undef CHAT
    return 0;
}

/* ------------------------------------------------------------------------------------ *
 * Exact optimum of the pipeline term sum_i c_i + (M-1) max_i c_i (Eq. 4 in its closed form) over the
 * partitions of one candidate.  For a limit t on the stage cost let f(t) be the smallest stage-cost sum
 * among partitions whose stages all cost at most t (additive recurrence, smallest split on ties).  The
 * optimum is reached at a limit that equals some stage cost, so the limits are swept upward from the
 * bottleneck B*: every pass reports the smallest stage cost it had to skip, which is the next limit.
 * With f_min = f(infinity), a partition whose largest stage costs t cannot beat the incumbent V once
 * f_min + (M-1) t >= V, which ends the sweep.  The first limit reaching the smallest value wins.
 * ------------------------------------------------------------------------------------ */
typedef struct { int64_t sum, mx, next; int ok; uint8_t k[ORC_MAX_PP + 1]; } add_pass;

static void additive_pass(const stage_ctx *cx, int64_t limit, int64_t *D, uint8_t *CH, add_pass *out)
{
    const int N = cx->N, PP = cx->PP;
#define DAT(i, j) D[(size_t)(i) * (N + 1) + (j)]
#define CHAT(i, j) CH[(size_t)(i) * (N + 1) + (j)]
    for (int i = 0; i <= PP; ++i)
        for (int j = 0; j <= N; ++j) { DAT(i, j) = ORC_INF; CHAT(i, j) = 255; }
    DAT(0, 0) = 0;
    out->next = ORC_INF;
    for (int i = 1; i <= PP; ++i)
        for (int j = i; j <= N - PP + i; ++j)
            for (int k = i - 1; k <= j - 1; ++k) {
                int64_t c = ctx_stage_cost(cx, i, k, j, NULL);
                if (c >= ORC_INF) continue;
                if (c > limit) { if (c < out->next) out->next = c; continue; }   /* smallest skipped cost */
                if (DAT(i - 1, k) >= ORC_INF) continue;
                int64_t v = DAT(i - 1, k) + c;
                if (v < DAT(i, j)) { DAT(i, j) = v; CHAT(i, j) = (uint8_t)k; }
            }
    out->ok = DAT(PP, N) < ORC_INF;
    out->sum = DAT(PP, N);
    out->mx = 0;
    if (out->ok) {
        int j = N;
        out->k[PP] = (uint8_t)N;
        for (int i = PP; i >= 1; --i) {
            int k = CHAT(i, j);
            int64_t c = ctx_stage_cost(cx, i, k, j, NULL);
            if (c > out->mx) out->mx = c;
            out->k[i - 1] = (uint8_t)k;
            j = k;
        }
    }
#undef DAT
#undef CHAT
}

int orc_candidate_exact(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                        const int64_t *c2, const int64_t *coef, orc_result *res, int64_t *n_passes)
{
    const int N = pr->N, PP = pc->PP;
    orc_result first;
    int rc0 = orc_candidate(pr, pc, mp, rc_mask, c2, coef, &first, NULL, NULL);
    if (n_passes) *n_passes = 0;
    if (rc0 != 0) { *res = first; return rc0; }
    const int64_t Bstar = first.bottleneck, M1 = pc->M - 1;
    stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
    int64_t *D = (int64_t *)malloc(sizeof(int64_t) * (size_t)(PP + 1) * (N + 1));
    uint8_t *CH = (uint8_t *)malloc((size_t)(PP + 1) * (N + 1));
    if (!D || !CH || !cx) { free(D); free(CH); free(cx); return -1; }
    ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
    add_pass best, cur, unl;
    int64_t passes = 2;
    additive_pass(cx, Bstar, D, CH, &best);                 /* limit B*: the refinement */
    additive_pass(cx, ORC_INF - 1, D, CH, &unl);            /* no limit: f_min */
    int64_t Vbest = best.sum + M1 * best.mx;
    const int64_t fmin = unl.sum;
    int64_t t = best.next;
    while (t < ORC_INF && fmin + M1 * t < Vbest) {
        additive_pass(cx, t, D, CH, &cur);
        passes++;
        if (cur.ok && cur.sum + M1 * cur.mx < Vbest) { best = cur; Vbest = cur.sum + M1 * cur.mx; }
        t = cur.next;
    }
    if (unl.sum + M1 * unl.mx < Vbest) { best = unl; Vbest = unl.sum + M1 * unl.mx; }
    if (n_passes) *n_passes = passes;
    /* objective on the chosen partition */
    memset(res, 0, sizeof(*res));
    res->bottleneck = Bstar;
    int64_t sum = 0, mx = 0, tsync = 0, topt = 0;
    for (int i = 1; i <= PP; ++i) {
        int k = best.k[i - 1], j = best.k[i], r;
        int64_t c = ctx_stage_cost(cx, i, k, j, &r);
        res->n[i - 1] = (uint8_t)(j - k);
        res->r[i - 1] = (uint8_t)r;
        res->c[i - 1] = c;
        sum += c;
        if (c > mx) mx = c;
        unsigned mask = mp->mask[i - 1];
        int64_t sy = mask_max(pr, mask, coef, ORC_SLAT), op = 0;
        for (int l = k; l < j; ++l) {
            sy += mask_max(pr, mask, coef, ORC_SBW + pr->kind[l]);
            op += mask_max(pr, mask, coef, ORC_OPT + pr->kind[l]);
        }
        if (sy > tsync) tsync = sy;
        if (op > topt) topt = op;
    }
    res->T_pipe = sum + M1 * mx;
    res->T_sync = tsync;
    res->T_opt = topt;
    res->T_iter = res->T_pipe + tsync + topt;
    if (pruned_by_hetero_comm(pr, pc, mp, coef, sum, res->n)) res->T_iter = res->T_pipe = ORC_INF;
    free(D); free(CH); free(cx);
    return 0;
}

/* Exhaustive minimum of sum + (M-1) max over every contiguous partition (no recurrence, no memo). */
static void bf_pipe_rec(const stage_ctx *cx, int stage, int nstages, int start, int end, int64_t M1,
                        int64_t cur_sum, int64_t cur_max, int64_t *best)
{
    if (stage == nstages) {
        int64_t c = ctx_stage_cost(cx, stage, start, end, NULL);
        if (c >= ORC_INF) return;
        int64_t mx = c > cur_max ? c : cur_max, v = cur_sum + c + M1 * mx;
        if (v < *best) *best = v;
        return;
    }
    for (int cut = start + 1; cut <= end - (nstages - stage); ++cut) {
        int64_t c = ctx_stage_cost(cx, stage, start, cut, NULL);
        if (c >= ORC_INF) continue;
        bf_pipe_rec(cx, stage + 1, nstages, cut, end, M1, cur_sum + c, c > cur_max ? c : cur_max, best);
    }
}

int64_t orc_bruteforce_pipe(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                            const int64_t *c2, const int64_t *coef)
{
    int64_t best = ORC_INF;
    stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
    if (!cx) return -1;
    ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
    bf_pipe_rec(cx, 1, pc->PP, 0, pr->N, pc->M - 1, 0, 0, &best);
    free(cx);
    return best;
}

/* Exhaustive check of the refinement: smallest sum of stage costs over every contiguous partition of
 * layers 1..j into stages 1..i whose stages all cost at most `limit` (no recurrence, no memo). */
static void bf_sum_rec(const stage_ctx *cx, int stage, int nstages, int start, int end, int64_t limit,
                       int64_t cur_sum, int64_t *best)
{
    if (stage == nstages) {
        int64_t c = ctx_stage_cost(cx, stage, start, end, NULL);
        if (c <= limit && c < ORC_INF && cur_sum + c < *best) *best = cur_sum + c;
        return;
    }
    for (int cut = start + 1; cut <= end - (nstages - stage); ++cut) {
        int64_t c = ctx_stage_cost(cx, stage, start, cut, NULL);
        if (c > limit || c >= ORC_INF) continue;
        bf_sum_rec(cx, stage + 1, nstages, cut, end, limit, cur_sum + c, best);
    }
}

int64_t orc_bruteforce_sum(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                           const int64_t *c2, const int64_t *coef, int i, int j, int64_t limit)
{
    int64_t best = ORC_INF;
    if (i == 0) return j == 0 ? 0 : ORC_INF;
    if (j >= i) {
        stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
        if (!cx) return -1;
        ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
        bf_sum_rec(cx, 1, i, 0, j, limit, 0, &best);
        free(cx);
    }
    return best;
}

/* Exhaustive minimum over every contiguous partition of layers 1..j into stages 1..i of the
 * largest stage cost (no recurrence, no memo): the plain definition of the bottleneck. */
static void bf_rec(const stage_ctx *cx, int stage, int nstages, int start, int end,
                   int64_t cur_max, int64_t *best, uint64_t *count)
{
    if (stage == nstages) {
        int64_t c = ctx_stage_cost(cx, stage, start, end, NULL);
        int64_t v = c > cur_max ? c : cur_max;
        if (v < *best) *best = v;
        (*count)++;
        return;
    }
    /* leave at least one layer for each later stage */
    for (int cut = start + 1; cut <= end - (nstages - stage); ++cut) {
        int64_t c = ctx_stage_cost(cx, stage, start, cut, NULL);
        int64_t v = c > cur_max ? c : cur_max;
        bf_rec(cx, stage + 1, nstages, cut, end, v, best, count);
    }
}

int64_t orc_bruteforce(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                       const int64_t *c2, const int64_t *coef, int i, int j, uint64_t *n_partitions)
{
    int64_t best = ORC_INF;
    uint64_t count = 0;
    if (i == 0) { if (n_partitions) *n_partitions = 0; return j == 0 ? 0 : ORC_INF; }
    if (j >= i) {
        stage_ctx *cx = (stage_ctx *)malloc(sizeof(stage_ctx));
        if (!cx) return -1;
        ctx_build(cx, pr, pc, mp, rc_mask, c2, coef);
        bf_rec(cx, 1, i, 0, j, 0, &best, &count);
        free(cx);
    }
    if (n_partitions) *n_partitions = count;
    return best > ORC_INF ? ORC_INF : best;
}

/* ------------------------------------------------------------------------------------ *
 * Candidate index -> evaluation; exhaustive search with (cost, index) argmin.
 * ------------------------------------------------------------------------------------ */
static int64_t find_pconf(const orc_pconf *pcs, uint64_t n_pconf, uint64_t n_rc, uint64_t index)
{
    for (uint64_t p = 0; p < n_pconf; ++p)
        if (index >= pcs[p].offset && index < pcs[p].offset + pcs[p].nmap * n_rc) return (int64_t)p;
    return -1;
}

int orc_eval_index(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t index,
                   orc_plan *out, int64_t *dp_table, uint8_t *ch_table)
{
    int64_t p = find_pconf(pcs, n_pconf, (uint64_t)pr->n_rc, index);
    if (p < 0) return -1;
    const orc_pconf *pc = &pcs[p];
    uint64_t local = index - pc->offset;
    uint64_t map_idx = local / (uint64_t)pr->n_rc, rc_idx = local % (uint64_t)pr->n_rc;
    int64_t *c2 = (int64_t *)malloc(sizeof(int64_t) * (size_t)pr->T * pr->N * 2);
    int64_t coef[ORC_MAX_TYPES * ORC_NCOEF];
    if (!c2) return -1;
    orc_layer_costs(pr, pc, c2, NULL, coef, NULL);
    memset(out, 0, sizeof(*out));
    out->index = index;
    out->pc = *pc;
    out->rc_mask = pr->rc_masks[rc_idx];
    int rcode = orc_decode(pr, pc, map_idx, &out->map);
    if (rcode == 0) rcode = orc_candidate(pr, pc, &out->map, out->rc_mask, c2, coef, &out->res, dp_table, ch_table);
    free(c2);
    return rcode < 0 ? rcode : 0;
}

int orc_search(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t first, uint64_t count,
               int64_t *costs, int64_t *bottlenecks, orc_plan *best, uint64_t *n_feasible)
{
    int64_t *c2 = (int64_t *)malloc(sizeof(int64_t) * (size_t)pr->T * pr->N * 2);
    int64_t coef[ORC_MAX_TYPES * ORC_NCOEF];
    int64_t best_cost = ORC_INF;
    uint64_t feas = 0;
    if (!c2) return -1;
    if (best) { memset(best, 0, sizeof(*best)); best->res.T_iter = ORC_INF; best->index = UINT64_MAX; }
    for (uint64_t p = 0; p < n_pconf; ++p) {
        const orc_pconf *pc = &pcs[p];
        uint64_t lo = pc->offset, hi = pc->offset + pc->nmap * (uint64_t)pr->n_rc;
        if (hi <= first || lo >= first + count) continue;
        orc_layer_costs(pr, pc, c2, NULL, coef, NULL);
        for (uint64_t map_idx = 0; map_idx < pc->nmap; ++map_idx) {
            orc_mapping mp;
            int decoded = 0;
            for (int rc = 0; rc < pr->n_rc; ++rc) {
                uint64_t idx = lo + map_idx * (uint64_t)pr->n_rc + (uint64_t)rc;
                if (idx < first || idx >= first + count) continue;
                if (!decoded) { orc_decode(pr, pc, map_idx, &mp); decoded = 1; }
                orc_result res;
                orc_candidate(pr, pc, &mp, pr->rc_masks[rc], c2, coef, &res, NULL, NULL);
                if (costs) costs[idx - first] = res.T_iter;
                if (bottlenecks) bottlenecks[idx - first] = res.bottleneck;
                if (res.T_iter < ORC_INF) feas++;
                if (res.T_iter < best_cost) {           /* ascending index + strict: lowest index wins */
                    best_cost = res.T_iter;
                    if (best) {
                        best->index = idx; best->pc = *pc; best->map = mp;
                        best->rc_mask = pr->rc_masks[rc]; best->res = res;
                    }
                }
            }
        }
    }
    if (n_feasible) *n_feasible = feas;
    free(c2);
    return 0;
}

/* Timing harness: evaluates every candidate of configurations p_first, p_first+stride, ...
 * (threads > 1 spreads configurations over OpenMP threads; the per-candidate work is the
 * plain code above).  Returns the (cost, index) minimum over what it evaluated. */
static int g_refine = 0;    /* evaluation mode of the whole-space harnesses below: 0 plain, 1 refined, 2 exact pipeline term */
void orc_set_refine(int on) { g_refine = on; }

int orc_search_pconfs(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t p_first,
                      uint64_t p_stride, uint64_t *n_done, int64_t *best_cost, uint64_t *best_index,
                      int64_t *costs, int64_t *bottlenecks)
{
    return orc_search_pconfs_plans(pr, pcs, n_pconf, p_first, p_stride, n_done, best_cost, best_index, costs, bottlenecks,
                                   NULL, NULL);
}

/* the same, also returning every candidate's partition (layers per stage) and recomputation levels,
 * [n_cand][ORC_MAX_PP] each, zero for infeasible candidates */
int orc_search_pconfs_plans(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t p_first,
                            uint64_t p_stride, uint64_t *n_done, int64_t *best_cost, uint64_t *best_index,
                            int64_t *costs, int64_t *bottlenecks, uint8_t *parts, uint8_t *levels)
{
    int64_t gbest = ORC_INF;
    uint64_t gidx = UINT64_MAX, done = 0;
    if (p_stride == 0) p_stride = 1;
    int64_t nsel = p_first < n_pconf ? (int64_t)((n_pconf - p_first + p_stride - 1) / p_stride) : 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : done)
    for (int64_t q = 0; q < nsel; ++q) {
        uint64_t p = p_first + (uint64_t)q * p_stride;
        const orc_pconf *pc = &pcs[p];
        int64_t *c2 = (int64_t *)malloc(sizeof(int64_t) * (size_t)pr->T * pr->N * 2);
        int64_t coef[ORC_MAX_TYPES * ORC_NCOEF];
        int64_t lbest = ORC_INF;
        uint64_t lidx = UINT64_MAX;
        orc_layer_costs(pr, pc, c2, NULL, coef, NULL);
        for (uint64_t map_idx = 0; map_idx < pc->nmap; ++map_idx) {
            orc_mapping mp;
            orc_decode(pr, pc, map_idx, &mp);
            for (int rc = 0; rc < pr->n_rc; ++rc) {
                orc_result res;
                if (g_refine == 2) orc_candidate_exact(pr, pc, &mp, pr->rc_masks[rc], c2, coef, &res, NULL);
                else if (g_refine) orc_candidate_refined(pr, pc, &mp, pr->rc_masks[rc], c2, coef, &res);
                else orc_candidate(pr, pc, &mp, pr->rc_masks[rc], c2, coef, &res, NULL, NULL);
                uint64_t idx = pc->offset + map_idx * (uint64_t)pr->n_rc + (uint64_t)rc;
                if (costs) costs[idx] = res.T_iter;              /* indexed by candidate, whole space */
                if (bottlenecks) bottlenecks[idx] = res.bottleneck;
                if (parts) memcpy(parts + idx * ORC_MAX_PP, res.n, ORC_MAX_PP);
                if (levels) memcpy(levels + idx * ORC_MAX_PP, res.r, ORC_MAX_PP);
                if (res.T_iter < lbest) { lbest = res.T_iter; lidx = idx; }
                done++;
            }
        }
        free(c2);
#pragma omp critical
        {
            if (lbest < gbest || (lbest == gbest && lidx < gidx)) { gbest = lbest; gidx = lidx; }
        }
    }
    *n_done = done;
    *best_cost = gbest;
    *best_index = gidx;
    return 0;
}


/* ==================================================================================== *
 * fp64 mode: the same definitions with the layer costs and time coefficients kept as doubles
 * (no rounding to integer ns); the memory test stays on the integer byte coefficients, the
 * recomputation time factor is tau_q / 1024.0 and an infeasible cost is +infinity.
 * ==================================================================================== */
typedef struct {
    int N, PP, R;
    int64_t M;
    uint32_t rc_mask;
    const int32_t *xi_q, *tau_q;
    double PF[ORC_MAX_PP][ORC_MAX_N + 1], PB[ORC_MAX_PP][ORC_MAX_N + 1];
    int64_t PW[ORC_MAX_N + 1], PA[ORC_MAX_N + 1];
    int32_t PK[ORC_MAX_N + 1];
    int64_t cap[ORC_MAX_PP], mpre, mpost, mx;
    double K[ORC_MAX_PP];
    int32_t nmin[ORC_MAX_PP], nmax[ORC_MAX_PP];
} stage_ctx_f;

static double mask_max_f(const orc_problem *pr, unsigned mask, const double *coeff, int q)
{
    double best = 0.0;
    int seen = 0;
    for (int h = 0; h < pr->T; ++h)
        if (mask & (1u << h)) {
            double x = coeff[h * ORC_NCOEF + q];
            if (!seen || x > best) best = x;
            seen = 1;
        }
    return best;
}

static void ctx_build_f(stage_ctx_f *cx, const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                        uint32_t rc_mask, const double *c2f, const int64_t *coef, const double *coeff)
{
    const int N = pr->N, PP = pc->PP;
    cx->N = N; cx->PP = PP; cx->R = pr->R; cx->M = pc->M; cx->rc_mask = rc_mask;
    cx->xi_q = pr->xi_q; cx->tau_q = pr->tau_q;
    orc_window(pr, pc, mp, cx->nmin, cx->nmax);
    cx->PW[0] = cx->PA[0] = 0; cx->PK[0] = 0;
    for (int l = 0; l < N; ++l) {
        cx->PW[l + 1] = cx->PW[l] + coef[ORC_MW + pr->kind[l]];
        cx->PA[l + 1] = cx->PA[l] + coef[ORC_MA + pr->kind[l]];
        cx->PK[l + 1] = cx->PK[l] + (pr->kind[l] == ORC_MOE ? 1 : 0);
    }
    cx->mpre = coef[ORC_MPRE]; cx->mpost = coef[ORC_MPOST]; cx->mx = coef[ORC_MX];
    for (int s = 0; s < PP; ++s) {
        const unsigned mask = mp->mask[s];
        const int i = s + 1;
        cx->PF[s][0] = cx->PB[s][0] = 0.0;
        for (int l = 0; l < N; ++l) {
            double F = 0.0, Bk = 0.0;
            int seen = 0;
            for (int h = 0; h < pr->T; ++h)
                if (mask & (1u << h)) {
                    double qf = c2f[((int64_t)h * N + l) * 2], qb = c2f[((int64_t)h * N + l) * 2 + 1];
                    if (!seen || qf > F) F = qf;
                    if (!seen || qb > Bk) Bk = qb;
                    seen = 1;
                }
            cx->PF[s][l + 1] = cx->PF[s][l] + F;
            cx->PB[s][l + 1] = cx->PB[s][l] + Bk;
        }
        int64_t cap = 0;
        int seen = 0;
        for (int h = 0; h < pr->T; ++h)
            if (mask & (1u << h)) {
                if (!seen || pr->cap_eff[h] < cap) cap = pr->cap_eff[h];
                seen = 1;
            }
        cx->cap[s] = cap;
        double K = 0.0;
        if (i == 1) K += mask_max_f(pr, mask, coeff, ORC_KPRE);
        if (i == PP) K += mask_max_f(pr, mask, coeff, ORC_KPOST);
        if (i > 1) {
            int hb = mp->hb[s], ha = mp->ha[s];
            if (mp->cls[s] == ORC_INTRA) K += coeff[hb * ORC_NCOEF + ORC_KP2P_INTRA];
            else if (mp->cls[s] == ORC_INTER) K += coeff[hb * ORC_NCOEF + ORC_KP2P_INTER];
            else K += coeff[hb * ORC_NCOEF + ORC_KP2P_CROSS + ha];
        }
        cx->K[s] = K;
    }
}

static double ctx_stage_cost_f(const stage_ctx_f *cx, int i, int a, int b, int *r_out)
{
    const int s = i - 1, PP = cx->PP;
    if (r_out) *r_out = -1;
    const int n = b - a;
    if (n < cx->nmin[s] || n > cx->nmax[s]) return INFINITY;
    const int has_moe = cx->PK[b] - cx->PK[a] > 0;
    const int64_t Wb = (cx->PW[b] - cx->PW[a]) + (i == 1 ? cx->mpre : 0) + (i == PP ? cx->mpost : 0)
                       + (has_moe ? cx->mx : 0);
    const int64_t Mstore = cx->M < PP - i + 1 ? cx->M : PP - i + 1;
    const int64_t A = Mstore * (cx->PA[b] - cx->PA[a]);
    int rstar = -1;
    for (int r = 0; r < cx->R && rstar < 0; ++r)
        if ((cx->rc_mask >> r) & 1u)
            if (Wb + ((int64_t)cx->xi_q[r] * A) / 1024 <= cx->cap[s]) rstar = r;
    if (rstar < 0) return INFINITY;
    if (r_out) *r_out = rstar;
    const double SF = cx->PF[s][b] - cx->PF[s][a], SB = cx->PB[s][b] - cx->PB[s][a];
    return SF + SB + ((double)cx->tau_q[rstar] / 1024.0) * SF + cx->K[s];
}

int orc_candidate_f64(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                      const double *c2f, const int64_t *coef, const double *coeff, orc_result_f *res)
{
    const int N = pr->N, PP = pc->PP;
    stage_ctx_f *cx = (stage_ctx_f *)malloc(sizeof(stage_ctx_f));
    double *DPt = (double *)malloc(sizeof(double) * (size_t)(PP + 1) * (N + 1));
    uint8_t *CH = (uint8_t *)malloc((size_t)(PP + 1) * (N + 1));
    if (!DPt || !CH || !cx) { free(DPt); free(CH); free(cx); return -1; }
    ctx_build_f(cx, pr, pc, mp, rc_mask, c2f, coef, coeff);
#define DPAT(i, j) DPt[(size_t)(i) * (N + 1) + (j)]
#define CHAT(i, j) CH[(size_t)(i) * (N + 1) + (j)]
    for (int i = 0; i <= PP; ++i)
        for (int j = 0; j <= N; ++j) { DPAT(i, j) = INFINITY; CHAT(i, j) = 255; }
    DPAT(0, 0) = 0.0;
    for (int i = 1; i <= PP; ++i)
        for (int j = i; j <= N - PP + i; ++j)
            for (int k = i - 1; k <= j - 1; ++k) {
                if (!(DPAT(i - 1, k) < INFINITY)) continue;
                double c = ctx_stage_cost_f(cx, i, k, j, NULL);
                double v = DPAT(i - 1, k) > c ? DPAT(i - 1, k) : c;
                if (v < DPAT(i, j)) { DPAT(i, j) = v; CHAT(i, j) = (uint8_t)k; }
            }
    memset(res, 0, sizeof(*res));
    res->bottleneck = DPAT(PP, N);
    if (!(res->bottleneck < INFINITY)) {
        res->T_iter = res->T_pipe = INFINITY;
        free(DPt); free(CH); free(cx);
        return 1;
    }
    double sum = 0.0, mx = 0.0, tsync = 0.0, topt = 0.0;
    int j = N;
    for (int i = PP; i >= 1; --i) {
        int k = CHAT(i, j), r;
        double c = ctx_stage_cost_f(cx, i, k, j, &r);
        res->n[i - 1] = (uint8_t)(j - k);
        res->r[i - 1] = (uint8_t)r;
        res->c[i - 1] = c;
        if (c > mx) mx = c;
        unsigned mask = mp->mask[i - 1];
        double sy = mask_max_f(pr, mask, coeff, ORC_SLAT), op = 0.0;
        for (int l = k; l < j; ++l) {
            sy += mask_max_f(pr, mask, coeff, ORC_SBW + pr->kind[l]);
            op += mask_max_f(pr, mask, coeff, ORC_OPT + pr->kind[l]);
        }
        if (sy > tsync) tsync = sy;
        if (op > topt) topt = op;
        j = k;
    }
    for (int i = 0; i < PP; ++i) sum += res->c[i];          /* stage 1 .. PP */
    res->T_pipe = sum + (double)(pc->M - 1) * mx;
    res->T_sync = tsync;
    res->T_opt = topt;
    res->T_iter = res->T_pipe + tsync + topt;
    if (pr->eta_q > 0) {                                   /* Pruning 3 on the unrounded values */
        double th = 0.0;
        for (int st = 1; st < PP; ++st)
            if (mp->cls[st] == ORC_CROSS) th += coeff[mp->hb[st] * ORC_NCOEF + ORC_KP2P_CROSS + mp->ha[st]];
        if (pr->het_coll) {                                /* mixed-type stages: dispatch and combine on the cross-type link */
            int a = 0;
            for (int st = 0; st < PP; ++st) {
                const unsigned mask = mp->mask[st];
                if (mask & (mask - 1)) {
                    int n_moe = 0;
                    for (int l = a; l < a + res->n[st]; ++l) n_moe += pr->kind[l] == ORC_MOE;
                    th += (double)n_moe * mask_max_f(pr, mask, coeff, ORC_KXD);
                }
                a += res->n[st];
            }
        }
        if (th * (double)PP * 1024.0 > (double)pr->eta_q * sum) res->T_iter = res->T_pipe = INFINITY;
    }
    free(DPt); free(CH); free(cx);
#undef DPAT
#undef CHAT
    return 0;
}

/* every candidate of every p_stride-th configuration in fp64 mode (OpenMP over configurations);
 * costs / bottlenecks are indexed by candidate over the whole space, partitions as [n_cand][ORC_MAX_PP] */
int orc_search_pconfs_f64(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t p_first,
                          uint64_t p_stride, uint64_t *n_done, double *costs, double *bottlenecks, uint8_t *parts)
{
    uint64_t done = 0;
    if (p_stride == 0) p_stride = 1;
    int64_t nsel = p_first < n_pconf ? (int64_t)((n_pconf - p_first + p_stride - 1) / p_stride) : 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : done)
    for (int64_t q = 0; q < nsel; ++q) {
        uint64_t p = p_first + (uint64_t)q * p_stride;
        const orc_pconf *pc = &pcs[p];
        double *c2f = (double *)malloc(sizeof(double) * (size_t)pr->T * pr->N * 2);
        int64_t coef[ORC_MAX_TYPES * ORC_NCOEF];
        double coeff[ORC_MAX_TYPES * ORC_NCOEF];
        orc_layer_costs(pr, pc, NULL, c2f, coef, coeff);
        for (uint64_t map_idx = 0; map_idx < pc->nmap; ++map_idx) {
            orc_mapping mp;
            orc_decode(pr, pc, map_idx, &mp);
            for (int rc = 0; rc < pr->n_rc; ++rc) {
                orc_result_f res;
                orc_candidate_f64(pr, pc, &mp, pr->rc_masks[rc], c2f, coef, coeff, &res);
                uint64_t idx = pc->offset + map_idx * (uint64_t)pr->n_rc + (uint64_t)rc;
                if (costs) costs[idx] = res.T_iter;
                if (bottlenecks) bottlenecks[idx] = res.bottleneck;
                if (parts) memcpy(parts + idx * ORC_MAX_PP, res.n, ORC_MAX_PP);
                done++;
            }
        }
        free(c2f);
    }
    *n_done = done;
    return 0;
}


/* ==================================================================================== *
 * Joint recurrence over the device state (the form printed in Sec. 3.5 / Algorithm 1, with the
 * min-max objective used throughout this library): DP[j][u][t] = smallest achievable largest
 * stage cost when the first |u| stages hold the first j layers, u[h] of them run on device type h
 * and the last one on type t.  It replaces the enumeration of stage-type sequences: the value at
 * u = (all stages placed), j = N is the minimum over ALL sequences of the per-sequence bottleneck.
 * Defined for configurations whose stages are homogeneous (G divides every m_h).
 * ==================================================================================== */
static int64_t joint_stage_cost(const orc_problem *pr, const orc_pconf *pc, uint32_t rc_mask, const int64_t *c2,
                                const int64_t *coef, const int32_t *nminT, const int32_t *nmaxT,
                                int i, int t, int tprev, int q, int a, int b)
{
    const int N = pr->N, PP = pc->PP;
    const int n = b - a;
    if (n < nminT[t] || n > nmaxT[t]) return ORC_INF;
    int64_t SF = 0, SB = 0, SW = 0, SA = 0;
    int has_moe = 0;
    for (int l = a; l < b; ++l) {
        SF += c2[((int64_t)t * N + l) * 2];
        SB += c2[((int64_t)t * N + l) * 2 + 1];
        SW += coef[ORC_MW + pr->kind[l]];
        SA += coef[ORC_MA + pr->kind[l]];
        if (pr->kind[l] == ORC_MOE) has_moe = 1;
    }
    const int64_t Mstore = pc->M < PP - i + 1 ? pc->M : PP - i + 1;
    const int64_t Wb = SW + (i == 1 ? coef[ORC_MPRE] : 0) + (i == PP ? coef[ORC_MPOST] : 0) + (has_moe ? coef[ORC_MX] : 0);
    const int64_t A = Mstore * SA;
    int rstar = -1;
    for (int r = 0; r < pr->R && rstar < 0; ++r)
        if ((rc_mask >> r) & 1u)
            if (Wb + ((int64_t)pr->xi_q[r] * A) / 1024 <= pr->cap_eff[t]) rstar = r;
    if (rstar < 0) return ORC_INF;
    int64_t K = 0;
    if (i == 1) K += coef[t * ORC_NCOEF + ORC_KPRE];
    if (i == PP) K += coef[t * ORC_NCOEF + ORC_KPOST];
    if (i > 1) {
        if (tprev != t) K += coef[t * ORC_NCOEF + ORC_KP2P_CROSS + tprev];
        else {
            /* q-th stage of its type (0-based): it starts at device q*G of the type's device line */
            const int64_t first = (int64_t)q * pc->G;
            const int same_node = (first - 1) / pr->node_size[t] == first / pr->node_size[t];
            K += coef[t * ORC_NCOEF + (same_node ? ORC_KP2P_INTRA : ORC_KP2P_INTER)];
        }
    }
    return SF + SB + ((int64_t)pr->tau_q[rstar] * SF) / 1024 + K;
}

/* returns the minimum bottleneck over all stage-type sequences, ORC_INF if none is feasible,
 * -1 if the configuration's stages are not homogeneous */
int64_t orc_joint_bottleneck(const orc_problem *pr, const orc_pconf *pc, uint32_t rc_mask,
                             const int64_t *c2, const int64_t *coef)
{
    const int N = pr->N, PP = pc->PP, T = pr->T;
    int64_t m[ORC_MAX_TYPES];
    type_counts(pr, m);
    int cnt[ORC_MAX_TYPES] = {0, 0, 0, 0}, stride[ORC_MAX_TYPES];
    int S = 1;
    for (int h = 0; h < T; ++h) {
        if (m[h] % pc->G != 0) return -1;
        cnt[h] = (int)(m[h] / pc->G);
    }
    for (int h = 0; h < ORC_MAX_TYPES; ++h) { stride[h] = S; S *= (h < T ? cnt[h] : 0) + 1; }
    /* window per type: every sequence has the same multiset of stages, hence the same total rate */
    int32_t nminT[ORC_MAX_TYPES], nmaxT[ORC_MAX_TYPES];
    int64_t Ps = 0;
    for (int h = 0; h < T; ++h) Ps += (int64_t)cnt[h] * pr->P[h];
    for (int h = 0; h < T; ++h) {
        int64_t lo = 1, hi = N - PP + 1;
        if (pr->uniform) { lo = N / PP; hi = (N + PP - 1) / PP; }
        else if (pr->delta_q >= 0) {
            lo = ((int64_t)(1024 - pr->delta_q) * pr->P[h] * N) / (1024 * Ps);
            int64_t num = (int64_t)(1024 + pr->delta_q) * pr->P[h] * N, den = 1024 * Ps;
            hi = (num + den - 1) / den;
            if (lo < 1) lo = 1;
            if (hi > N - PP + 1) hi = N - PP + 1;
        }
        nminT[h] = (int32_t)lo; nmaxT[h] = (int32_t)hi;
    }
    const size_t cells = (size_t)S * T * (N + 1);
    int64_t *D = (int64_t *)malloc(sizeof(int64_t) * cells);
    if (!D) return -2;
    for (size_t x = 0; x < cells; ++x) D[x] = ORC_INF;
#define JAT(ui, t, j) D[((size_t)(ui) * T + (t)) * (N + 1) + (j)]
    for (int i = 1; i <= PP; ++i)                       /* level = number of stages placed */
        for (int ui = 0; ui < S; ++ui) {
            int u[ORC_MAX_TYPES], tot = 0;
            for (int h = 0; h < ORC_MAX_TYPES; ++h) { u[h] = (ui / stride[h]) % ((h < T ? cnt[h] : 0) + 1); tot += u[h]; }
            if (tot != i) continue;
            for (int t = 0; t < T; ++t) {
                if (u[t] == 0) continue;                  /* the last stage is of type t */
                const int up = ui - stride[t];
                for (int j = i; j <= N - PP + i; ++j) {
                    int64_t best = ORC_INF;
                    if (i == 1) {
                        best = joint_stage_cost(pr, pc, rc_mask, c2, coef, nminT, nmaxT, 1, t, -1, 0, 0, j);
                    } else {
                        for (int tp = 0; tp < T; ++tp) {
                            const int utp = (up / stride[tp]) % (cnt[tp] + 1);
                            if (utp == 0) continue;       /* the prefix cannot end with a type it does not contain */
                            for (int k = i - 1; k <= j - 1; ++k) {
                                const int64_t pv = JAT(up, tp, k);
                                if (pv >= ORC_INF) continue;
                                const int64_t c = joint_stage_cost(pr, pc, rc_mask, c2, coef, nminT, nmaxT, i, t, tp,
                                                                   u[t] - 1, k, j);
                                const int64_t v = pv > c ? pv : c;
                                if (v < best) best = v;
                            }
                        }
                    }
                    JAT(ui, t, j) = best;
                }
            }
        }
    int64_t ans = ORC_INF;
    for (int t = 0; t < T; ++t)
        if (cnt[t] > 0 && JAT(S - 1, t, N) < ans) ans = JAT(S - 1, t, N);
#undef JAT
    free(D);
    return ans;
}

/* ------------------------------------------------------------------------------------ *
 * Appendix B: the steady-state term written with the bottleneck stage's index s_max, evaluated for a
 * given plan (layers and recomputation level per stage).  Plain loops over stages and layers.
 * ------------------------------------------------------------------------------------ */
int orc_appendix_b(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                   const int64_t *c2, const int64_t *coef, const uint8_t *n, const uint8_t *r, orc_appb_result *res)
{
    const int N = pr->N, PP = pc->PP;
    memset(res, 0, sizeof(*res));
    int total = 0;
    for (int s = 0; s < PP; ++s) { if (n[s] == 0) total = -100000; total += n[s]; }
    if (total != N) { res->T_iter = ORC_INF; return 1; }
    int64_t edge = 0, cmax = -1, fsum = 0, f_upto_max = 0, tsync = 0, topt = 0;
    int smax = 0, a = 0;
    for (int s = 0; s < PP; ++s) {
        const unsigned mask = mp->mask[s];
        const int i = s + 1, b = a + n[s];
        int64_t tf = 0, tb = 0;
        for (int l = a; l < b; ++l) {
            int64_t F = 0, Bk = 0;
            int seen = 0;
            for (int h = 0; h < pr->T; ++h)
                if (mask & (1u << h)) {
                    const int64_t qf = c2[((int64_t)h * N + l) * 2], qb = c2[((int64_t)h * N + l) * 2 + 1];
                    if (!seen || qf > F) F = qf;
                    if (!seen || qb > Bk) Bk = qb;
                    seen = 1;
                }
            tf += F; tb += Bk;
        }
        tb += ((int64_t)pr->tau_q[r[s]] * tf) / 1024;                 /* forward work repeated in the backward pass */
        if (i == 1) tb += mask_max(pr, mask, coef, ORC_KPRE);
        if (i == PP) tb += mask_max(pr, mask, coef, ORC_KPOST);
        if (i > 1) {
            const int hb = mp->hb[s], ha = mp->ha[s];
            if (mp->cls[s] == ORC_INTRA) tb += coef[hb * ORC_NCOEF + ORC_KP2P_INTRA];
            else if (mp->cls[s] == ORC_INTER) tb += coef[hb * ORC_NCOEF + ORC_KP2P_INTER];
            else tb += coef[hb * ORC_NCOEF + ORC_KP2P_CROSS + ha];
        }
        const int64_t c = tf + tb;
        edge += c;
        fsum += tf;
        if (c > cmax) { cmax = c; smax = i; f_upto_max = fsum; }       /* strict: the first bottleneck stage */
        int64_t sy = mask_max(pr, mask, coef, ORC_SLAT), op = 0;
        for (int l = a; l < b; ++l) {
            sy += mask_max(pr, mask, coef, ORC_SBW + pr->kind[l]);
            op += mask_max(pr, mask, coef, ORC_OPT + pr->kind[l]);
        }
        if (sy > tsync) tsync = sy;
        if (op > topt) topt = op;
        a = b;
    }
    int64_t steady = (int64_t)pc->M - smax - 1;
    if (steady < 0) steady = 0;
    res->T_edge = edge;
    res->T_middle = f_upto_max + steady * cmax;
    res->T_sync = tsync; res->T_opt = topt;
    res->s_max = smax;
    res->T_iter = res->T_edge + res->T_middle + tsync + topt;
    return 0;
}

/* ------------------------------------------------------------------------------------------
 * Event simulation of the 1F1B schedule for a GIVEN plan (Sec. 3.3: "the end-to-end iteration
 * latency under the 1F1B pipeline schedule", which Eq. 4 and Appendix B put in closed form).
 * Stage i (1-based) runs, strictly in this order: min(PP - i, M) warm-up forward passes, then
 * forward / backward pairs while forwards remain, then the backward passes that are left.
 * F(i, m) starts when stage i is free and F(i-1, m) has finished; B(i, m) starts when stage i is
 * free and B(i+1, m) has finished (on the last stage: when its own F(i, m) has).  A forward pass of
 * stage i takes t_f,i, a backward pass t_b,i, split as in Appendix B: t_f,i is the forward time of
 * the stage's layers (slowest member type per layer), t_b,i everything else of the stage cost
 * (backward time, recomputation at the stage's level, the stage constant with its transfer term), so
 * transfers take no time of their own.  T_pipe_sim is the time the last backward pass ends,
 * T_iter = T_pipe_sim + T_sync + T_opt; T_pipe_closed = sum_i c_i + (M-1) max_i c_i is Eq. 4's
 * pipeline term for the same plan.  Returns 1 and T_iter = ORC_INF when n does not partition the layers.
 * ------------------------------------------------------------------------------------------ */
int orc_simulate_1f1b(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                      const int64_t *c2, const int64_t *coef, const uint8_t *n, const uint8_t *r, orc_sim_result *res)
{
    const int N = pr->N, PP = pc->PP, M = pc->M;
    memset(res, 0, sizeof(*res));
    int total = 0;
    for (int s = 0; s < PP; ++s) { if (n[s] == 0) total = -100000; total += n[s]; }
    if (total != N || M < 1) { res->T_iter = ORC_INF; return 1; }
    int64_t tf[ORC_MAX_PP], tb[ORC_MAX_PP], csum = 0, cmax = 0, tsync = 0, topt = 0;
    int a = 0;
    for (int s = 0; s < PP; ++s) {
        const unsigned mask = mp->mask[s];
        const int i = s + 1, b = a + n[s];
        int64_t F = 0, B = 0;
        for (int l = a; l < b; ++l) {
            int64_t fl = 0, bl = 0;
            for (int h = 0; h < pr->T; ++h)
                if (mask & (1u << h)) {
                    const int64_t qf = c2[((int64_t)h * N + l) * 2], qb = c2[((int64_t)h * N + l) * 2 + 1];
                    if (qf > fl) fl = qf;
                    if (qb > bl) bl = qb;
                }
            F += fl; B += bl;
        }
        B += ((int64_t)pr->tau_q[r[s]] * F) / 1024;
        if (i == 1) B += mask_max(pr, mask, coef, ORC_KPRE);
        if (i == PP) B += mask_max(pr, mask, coef, ORC_KPOST);
        if (i > 1) {
            const int hb = mp->hb[s], ha = mp->ha[s];
            B += coef[hb * ORC_NCOEF + (mp->cls[s] == ORC_CROSS ? ORC_KP2P_CROSS + ha : (mp->cls[s] == ORC_INTER ? ORC_KP2P_INTER : ORC_KP2P_INTRA))];
        }
        tf[s] = F; tb[s] = B;
        csum += F + B;
        if (F + B > cmax) cmax = F + B;
        int64_t sy = mask_max(pr, mask, coef, ORC_SLAT), op = 0;
        for (int l = a; l < b; ++l) {
            sy += mask_max(pr, mask, coef, ORC_SBW + pr->kind[l]);
            op += mask_max(pr, mask, coef, ORC_OPT + pr->kind[l]);
        }
        if (sy > tsync) tsync = sy;
        if (op > topt) topt = op;
        a = b;
    }
    /* finish times of every pass; -1: not run yet */
    int64_t *Fd = (int64_t *)malloc(sizeof(int64_t) * (size_t)PP * M * 2), *Bd = Fd + (size_t)PP * M;
    if (!Fd) { res->T_iter = ORC_INF; return 1; }
    for (size_t q = 0; q < (size_t)PP * M * 2; ++q) Fd[q] = -1;
    int nf[ORC_MAX_PP], nb[ORC_MAX_PP];
    int64_t t_free[ORC_MAX_PP];
    for (int s = 0; s < PP; ++s) { nf[s] = nb[s] = 0; t_free[s] = 0; }
    long remaining = 2L * PP * M;
    while (remaining > 0) {
        long before = remaining;
        for (int s = 0; s < PP; ++s) {
            const int warm = PP - 1 - s < M ? PP - 1 - s : M;
            for (;;) {
                if (nb[s] == M) break;
                /* the stage's next pass in its fixed order */
                const int fwd = nf[s] < M && (nf[s] < warm || nf[s] - nb[s] == warm);
                int64_t dep;
                if (fwd) dep = s == 0 ? 0 : Fd[(size_t)(s - 1) * M + nf[s]];
                else dep = s == PP - 1 ? Fd[(size_t)s * M + nb[s]] : Bd[(size_t)(s + 1) * M + nb[s]];
                if (dep < 0) break;                                        /* its input has not been produced yet */
                const int64_t start = t_free[s] > dep ? t_free[s] : dep;
                if (fwd) { t_free[s] = start + tf[s]; Fd[(size_t)s * M + nf[s]] = t_free[s]; nf[s]++; }
                else { t_free[s] = start + tb[s]; Bd[(size_t)s * M + nb[s]] = t_free[s]; nb[s]++; }
                remaining--;
            }
        }
        if (remaining == before) { free(Fd); res->T_iter = ORC_INF; return 1; }   /* cannot happen: the schedule has no cycle */
    }
    int64_t end = 0;
    for (int s = 0; s < PP; ++s) if (t_free[s] > end) end = t_free[s];
    free(Fd);
    res->T_pipe_sim = end;
    res->T_pipe_closed = csum + (int64_t)(M - 1) * cmax;
    res->T_sync = tsync; res->T_opt = topt;
    res->T_iter = end + tsync + topt;
    return 0;
}

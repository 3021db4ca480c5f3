/*
 * CPU oracle of the HAPMoE planner hot path -- TEST INFRASTRUCTURE, not a product path.
 *
 * A plain, slow, single-threaded restatement of what the planner computes: the 6-D
 * enumeration, the MoE-aware layer cost (Eq. 2, Eq. 3, load-imbalance scaling), the stage
 * memory model with minimal feasible recomputation, the per-candidate min-max pipeline
 * partitioning recurrence, the 1F1B closed-form iteration latency (Eq. 4), the appendix's
 * steady-state expression and an event simulation of the 1F1B schedule for given plans, and the global argmin (Eq. 1).  Only the tests, the smoke check and the benchmark's CPU-baseline leg may
 * call it.  It shares no code with the CUDA library.
 *
 * Parity status: every function below is pinned by tests that do not go through this file's
 * own formulas (hand-computed cost terms, brute force over all contiguous partitions,
 * closed forms and invariants).  Nothing here is "parity unpinned".
 */
#ifndef HAP_ORACLE_H
#define HAP_ORACLE_H
#include <stdint.h>

#define ORC_MAX_TYPES 4
#define ORC_MAX_PP 32
#define ORC_MAX_N 255
#define ORC_MAX_RC 4
#define ORC_INF ((int64_t)1 << 62)

enum { ORC_DENSE = 0, ORC_MOE = 1 };
enum { ORC_INTRA = 0, ORC_INTER = 1, ORC_CROSS = 2 };
enum { ORC_MODE_MULTISET = 0, ORC_MODE_BLOCK = 1 };

/* stage-level coefficients per (configuration, device type), all rounded to int64 */
enum {
    ORC_KPRE = 0, ORC_KPOST = 1, ORC_KP2P_INTRA = 2, ORC_KP2P_INTER = 3,
    ORC_KP2P_CROSS = 4, /* +h' for the sending type, 4 entries */
    ORC_SLAT = 8, ORC_SBW = 9, /* +kind */ ORC_OPT = 11, /* +kind */
    ORC_MW = 13, /* +kind */ ORC_MA = 15, /* +kind */ ORC_MX = 17, ORC_MPRE = 18, ORC_MPOST = 19,
    ORC_KXD = 20, /* dispatch + combine of an MoE layer over the cross-type link (Pruning 3 with het_coll) */
    ORC_NCOEF = 21
};

typedef struct {
    /* model */
    int32_t N, S, H, E, k, n_shared, F_dense, F_exp, nq, nkv, V, GB;
    double beta;
    const uint8_t *kind;
    /* cluster */
    int32_t T;
    const int64_t *P, *C;
    const int32_t *node_size;
    const double *bw_intra;
    int32_t n_nodes;
    const int32_t *node_type;
    const double *node_bw_inter;
    /* profile */
    int32_t ntp, ncp, nmb, nep;
    const int32_t *tp_list, *cp_list, *mb_list, *ep_list;
    const double *tdf, *tdb, *tff, *tfb, *tpre, *tpost, *eta, *croute;
    double kappa;
    const double *alpha;
    double chi;
    const double *rho;
    double gamma, ovl_tp, ovl_cp, ovl_dp;
    const double *act_coef;
    double capf;
    const double *copt;
    const int64_t *cap_eff;
    int32_t R;
    const int32_t *xi_q, *tau_q;
    /* search options */
    int32_t npp, ntpe;
    const int32_t *pp_list, *tpe_list;
    int32_t tp_max, delta_q;
    uint64_t map_cap;
    int32_t n_rc;
    const uint32_t *rc_masks;
    int32_t eta_q;      /* Pruning 3 threshold eta in 1/1024; <= 0: off */
    int32_t uniform;    /* ablation: uniform layer split only (floor/ceil of N/PP layers per stage) */
    /* communication-primitive table: link efficiency by message size (0 sizes: efficiency 1 everywhere) */
    int32_t n_fsize;
    int32_t het_coll;   /* Pruning 3 also counts the dispatch / combine traffic of stages that span device types */
    const double *fsize;    /* [n_fsize] bytes, ascending */
    const double *feff;     /* [3][n_fsize] efficiency in (0, 1] of an intra-node / inter-node / cross-type link */
} orc_problem;

typedef struct {
    int32_t PP, TP, CP, DP, EP, TPE, b, M, EDP, G;
    int32_t itp, icp, ib, iep, mode, pad;
    uint64_t nmap, offset;
} orc_pconf;

typedef struct {
    int32_t PP;
    uint8_t mask[ORC_MAX_PP];   /* bit h set: stage overlaps device type h */
    uint8_t cls[ORC_MAX_PP];    /* link class of the boundary entering stage s (s >= 1) */
    uint8_t ha[ORC_MAX_PP];     /* type of the last device of stage s-1 */
    uint8_t hb[ORC_MAX_PP];     /* type of the first device of stage s */
} orc_mapping;

typedef struct {
    int64_t T_iter, bottleneck, T_pipe, T_sync, T_opt;
    uint8_t n[ORC_MAX_PP];   /* layers per stage */
    uint8_t r[ORC_MAX_PP];   /* recompute level per stage */
    int64_t c[ORC_MAX_PP];   /* stage cost of the chosen partition */
} orc_result;

typedef struct {
    uint64_t index;
    orc_pconf pc;
    orc_mapping map;
    uint32_t rc_mask;
    orc_result res;
} orc_plan;

int orc_enumerate(const orc_problem *pr, orc_pconf *out, uint64_t cap, uint64_t *n_pconf, uint64_t *n_cand);
uint64_t orc_multiset_count(const int32_t *cnt, int T, uint64_t sat);
int orc_unrank_multiset(const int32_t *cnt, int T, int PP, uint64_t idx, uint8_t *seq);
uint64_t orc_rank_multiset(const int32_t *cnt, int T, int PP, const uint8_t *seq);
int orc_decode(const orc_problem *pr, const orc_pconf *pc, uint64_t map_idx, orc_mapping *out);
int orc_layer_costs(const orc_problem *pr, const orc_pconf *pc, int64_t *c2, double *c2f,
                    int64_t *coef, double *coeff);
int64_t orc_stage_cost(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                       uint32_t rc_mask, const int64_t *c2, const int64_t *coef,
                       int i, int a, int b, int *r_out);
int orc_window(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, int32_t *nmin, int32_t *nmax);
int orc_candidate(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                  const int64_t *c2, const int64_t *coef, orc_result *res,
                  int64_t *dp_table, uint8_t *ch_table);
int64_t orc_bruteforce(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                       const int64_t *c2, const int64_t *coef, int i, int j, uint64_t *n_partitions);
int orc_eval_index(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t index,
                   orc_plan *out, int64_t *dp_table, uint8_t *ch_table);
int orc_search(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t first, uint64_t count,
               int64_t *costs, int64_t *bottlenecks, orc_plan *best, uint64_t *n_feasible);
int orc_search_pconfs(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t p_first,
                      uint64_t p_stride, uint64_t *n_done, int64_t *best_cost, uint64_t *best_index,
                      int64_t *costs, int64_t *bottlenecks);
int orc_search_pconfs_plans(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t p_first,
                            uint64_t p_stride, uint64_t *n_done, int64_t *best_cost, uint64_t *best_index,
                            int64_t *costs, int64_t *bottlenecks, uint8_t *parts, uint8_t *levels);

/* refinement: smallest sum of stage costs among the bottleneck-optimal partitions */
int orc_candidate_refined(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                          const int64_t *c2, const int64_t *coef, orc_result *res);
int64_t orc_bruteforce_sum(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                           const int64_t *c2, const int64_t *coef, int i, int j, int64_t limit);
void orc_set_refine(int on);
/* exact optimum of sum + (M-1) max over the partitions of a candidate */
int orc_candidate_exact(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                        const int64_t *c2, const int64_t *coef, orc_result *res, int64_t *n_passes);
int64_t orc_bruteforce_pipe(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                            const int64_t *c2, const int64_t *coef);

/* joint recurrence over the device state: minimum bottleneck over all stage-type sequences */
int64_t orc_joint_bottleneck(const orc_problem *pr, const orc_pconf *pc, uint32_t rc_mask,
                             const int64_t *c2, const int64_t *coef);

/* fp64 mode (no rounding of times to integer ns); see hap_oracle.c */
typedef struct {
    double T_iter, bottleneck, T_pipe, T_sync, T_opt;
    uint8_t n[ORC_MAX_PP], r[ORC_MAX_PP];
    double c[ORC_MAX_PP];
} orc_result_f;
int orc_candidate_f64(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp, uint32_t rc_mask,
                      const double *c2f, const int64_t *coef, const double *coeff, orc_result_f *res);
int orc_search_pconfs_f64(const orc_problem *pr, const orc_pconf *pcs, uint64_t n_pconf, uint64_t p_first,
                          uint64_t p_stride, uint64_t *n_done, double *costs, double *bottlenecks, uint8_t *parts);
/* Iteration latency of a GIVEN plan by the appendix's steady-state expression (Appendix B, with Eq. 4):
 *   T_iter = T_edge + T_middle + T_dp-sync + T_opt,  T_edge = sum_i (t_f,i + t_b,i),
 *   s_max = the (first) stage with the largest t_f,i + t_b,i,
 *   T_middle = sum_{i <= s_max} t_f,i + (M - s_max - 1) * max_i (t_f,i + t_b,i),
 * stages 1-based.  t_f,i is the forward time of the stage's layers (slowest member type per layer); t_b,i is
 * everything else of the stage cost (backward time, recomputation at the stage's level r_i, the stage constant),
 * so t_f,i + t_b,i is the stage cost of the min-max recurrence.  The multiplier of the steady-state term is taken
 * as max(0, M - s_max - 1).  n: layers per stage (sum N), r: recomputation level per stage.  Returns 0, or 1 and
 * T_iter = ORC_INF when n does not partition the N layers. */
typedef struct {
    int64_t T_iter, T_edge, T_middle, T_sync, T_opt;
    int32_t s_max, pad;
} orc_appb_result;
int orc_appendix_b(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                   const int64_t *c2, const int64_t *coef, const uint8_t *n, const uint8_t *r, orc_appb_result *res);

/* Event simulation of the 1F1B schedule for a GIVEN plan (the schedule Eq. 4 and Appendix B put in closed form): the
 * time at which the last backward pass ends when every stage runs its passes in the 1F1B order (min(PP - i, M)
 * warm-up forwards, forward / backward pairs, remaining backwards), a forward pass of stage i taking t_f,i and a
 * backward pass t_b,i (split as for orc_appendix_b).  T_pipe_closed is Eq. 4's pipeline term for the same plan. */
typedef struct {
    int64_t T_iter, T_pipe_sim, T_pipe_closed, T_sync, T_opt;
} orc_sim_result;
int orc_simulate_1f1b(const orc_problem *pr, const orc_pconf *pc, const orc_mapping *mp,
                      const int64_t *c2, const int64_t *coef, const uint8_t *n, const uint8_t *r, orc_sim_result *res);

#endif

/*
 * libhap -- C ABI of the HAPMoE planner hot path on one NVIDIA B200 (sm_100a).
 *
 * The library evaluates the paper's MoE-aware cost model over the 6-D parallel space
 * (DP, PP, TP, CP, EP, TPE) x device-group-to-stage mappings x recomputation policies,
 * runs the per-candidate non-uniform pipeline-partitioning dynamic program under per-stage
 * memory feasibility and returns the argmin plan (problem statement: Sec. 3.2, Eq. 1).
 *
 * Conventions
 *  - Every function returns a hap_status; nothing throws, exits or prints.
 *  - Descriptor structs and the arrays they point to are HOST memory owned by the caller;
 *    hap_problem_create copies them, so they may be freed right after it returns.
 *  - Arguments named dev_* are DEVICE pointers owned by the caller (for example the
 *    data_ptr() of a torch tensor) on the device that was current at hap_problem_create.
 *    The library never frees or reallocates them.  Nullable ones are marked.
 *  - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Kernels are
 *    enqueued on it and the call returns without waiting, except where a function returns
 *    host values: that function synchronises `stream` (only that stream) before returning.
 *  - A hap_problem is not thread safe; use one per thread or serialise calls.
 *  - Times are nanoseconds, memory is bytes, both as int64 after round-to-nearest-even of
 *    the fp64 formula value ("integer mode").  HAP_INF marks an infeasible candidate.
 *  - Value limits (so that every sum stays below 2^62): global batch x layers <= 2^22, a layer's
 *    forward or backward time < 2^36 ns, a stage constant < 2^40 ns.  A violation found on the device is
 *    reported as HAP_E_RANGE by the next call that synchronises (hap_search_*, hap_count_cells,
 *    hap_get_timings); asynchronous calls cannot report it themselves.
 */
#ifndef HAP_H
#define HAP_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define HAP_MAX_TYPES 4      /* device types |H| */
#define HAP_MAX_PP 32        /* pipeline stages */
#define HAP_MAX_LAYERS 255   /* N */
#define HAP_MAX_RC 4         /* recomputation levels R */
#define HAP_MAX_RC_MASKS 8   /* recomputation policies n_rc */
#define HAP_MAX_LIST 16      /* entries of any degree list */
#define HAP_INF ((int64_t)1 << 62)

typedef enum {
    HAP_OK = 0,
    HAP_E_INVALID = 1,     /* bad descriptor or argument */
    HAP_E_NOMEM = 2,       /* host or device allocation failed */
    HAP_E_CUDA = 3,        /* a CUDA call failed; see hap_last_error */
    HAP_E_RANGE = 4,       /* index range outside the candidate space, or a cost overflowed */
    HAP_E_STATE = 5,       /* call order violated (e.g. hap_pipeline_dp before hap_enumerate) */
    HAP_E_INFEASIBLE = 6   /* every candidate violates the memory constraint of Eq. 1 */
} hap_status;

enum { HAP_DENSE = 0, HAP_MOE = 1 };                  /* layer kind */
enum { HAP_INTRA = 0, HAP_INTER = 1, HAP_CROSS = 2 }; /* link class (Sec. 3.3: intra-node, inter-node, cross-type) */
enum { HAP_MAP_MULTISET = 0, HAP_MAP_BLOCK = 1 };     /* mapping mode of a configuration */

/* Column layout of the per-(configuration, device type) stage coefficient row. */
enum {
    HAP_KPRE = 0,        /* embedding work charged to the first stage, ns */
    HAP_KPOST = 1,       /* LM head + loss work charged to the last stage, ns */
    HAP_KP2P_INTRA = 2,  /* activation + gradient transfer into a stage over an intra-node link, ns */
    HAP_KP2P_INTER = 3,  /* same, inter-node link between devices of one type */
    HAP_KP2P_CROSS = 4,  /* same, cross-type link; +h' where h' is the sending type (4 entries) */
    HAP_SLAT = 8,        /* latency part of T_dp-sync, ns */
    HAP_SBW = 9,         /* bandwidth part of T_dp-sync per layer; +kind */
    HAP_OPT = 11,        /* T_opt per layer; +kind */
    HAP_MW = 13,         /* weights + gradients + optimizer state per layer, bytes; +kind */
    HAP_MA = 15,         /* activation bytes per layer per stored micro-batch; +kind */
    HAP_MX = 17,         /* M_moe-extra of a stage that holds at least one MoE layer, bytes */
    HAP_MPRE = 18,       /* embedding weights on the first stage, bytes */
    HAP_MPOST = 19,      /* LM head weights on the last stage, bytes */
    HAP_KXD = 20,        /* dispatch + combine of one MoE layer, forward and backward, when the expert-parallel group spans
                            device types: Eq. 3's volumes over the cross-type link class at chi x the type's inter-node
                            bandwidth, with the imbalance factor of Eq. 2, ns; read by Pruning 3 under
                            HAP_OPT_HETERO_DISPATCH only */
    HAP_NCOEF = 21
};

/* Model and training hyper-parameters (Sec. 3.2 "Input": N, S, H, E, k, batch sizes). */
typedef struct {
    int32_t N;          /* layers, 1..HAP_MAX_LAYERS */
    int32_t S;          /* sequence length */
    int32_t H;          /* hidden size */
    int32_t E;          /* routed experts per MoE layer */
    int32_t k;          /* top-k */
    int32_t n_shared;   /* shared experts per MoE layer */
    int32_t F_dense;    /* FFN width of dense layers */
    int32_t F_exp;      /* FFN width of one expert */
    int32_t nq, nkv;    /* attention heads / KV heads */
    int32_t V;          /* vocabulary */
    int32_t GB;         /* global batch (sequences) */
    double beta;        /* bytes per activation element */
    const uint8_t *kind; /* [N] HAP_DENSE / HAP_MOE */
} hap_model;

/* Cluster: device-type triples (P_h, C_h, B_h) and inventory {m_h} as a node list. */
typedef struct {
    int32_t n_types;               /* 1..HAP_MAX_TYPES; every type must own at least one node */
    const int64_t *P;              /* [n_types] peak GFLOP/s (used by the load-balance window) */
    const int64_t *C;              /* [n_types] raw memory capacity, bytes (informational) */
    const int32_t *node_size;      /* [n_types] devices per node of the type */
    const double *bw_intra;        /* [n_types] bytes/ns inside a node */
    int32_t n_nodes;
    const int32_t *node_type;      /* [n_nodes] type id of each node; a type's device line lists its nodes in this order */
    const double *node_bw_inter;   /* [n_nodes] bytes/ns of the node's uplink; a type uses the minimum over its nodes */
} hap_cluster;

/* Profiled lookup tables and calibrated coefficients (Sec. 3.3 and 3.4: compute table,
 * communication primitive table, memory calibration).  Table layout: row-major
 * [type][itp][icp][ib][layer] for the per-layer tables, [type][itp][icp][ib] for tpre/tpost,
 * where itp/icp/ib index tp_list/cp_list/mb_list. */
typedef struct {
    int32_t ntp, ncp, nmb, nep;
    const int32_t *tp_list, *cp_list, *mb_list, *ep_list;
    const double *tdf, *tdb;     /* t_dense forward / backward of one micro-batch, ns */
    const double *tff, *tfb;     /* t_ffn forward / backward (the part the experts replace), ns */
    const double *tpre, *tpost;  /* embedding / LM-head+loss forward+backward, ns */
    const double *eta;           /* [n_types] device-efficiency factor of Eq. 2, in (0,1] */
    const double *croute;        /* [n_types] router cost, ns per token*hidden element */
    double kappa;                /* the numerator constant of Eq. 2's expert term ("2" as printed) */
    const double *alpha;         /* [3] latency per collective step for HAP_INTRA/INTER/CROSS, ns */
    double chi;                  /* bandwidth factor of a cross-type link */
    const double *rho;           /* [nep] load imbalance (max expert load / mean load), >= 1 */
    double gamma;                /* imbalance weight in [0,1] */
    double ovl_tp, ovl_cp, ovl_dp; /* exposed fraction of TP / CP / DP collectives */
    const double *act_coef;      /* [2] activation bytes per token*hidden element, by layer kind */
    double capf;                 /* capacity factor of the dispatch buffers */
    const double *copt;          /* [n_types] optimizer time, ns per parameter */
    const int64_t *cap_eff;      /* [n_types] usable memory after calibration, bytes */
    int32_t R;                   /* recomputation levels, 1..HAP_MAX_RC; level 0 = none */
    const int32_t *xi_q;         /* [R] activation-memory factor xi(r) in 1/1024 */
    const int32_t *tau_q;        /* [R] fraction of the forward pass re-executed, in 1/1024 */
    /* Communication-primitive table (Sec. 3.4, "f_prim across link types"): the profiled efficiency of a link by
     * message size.  The volume term of every primitive (ring collectives, all-to-all / all-gather dispatch, p2p,
     * gradient sync), volume / bandwidth, is divided by the efficiency of its link class at its volume, piecewise
     * linear between the profiled sizes and constant outside them.  n_fsize = 0: no table, efficiency 1. */
    int32_t n_fsize;             /* 0..HAP_MAX_LIST profiled message sizes */
    const double *fsize;         /* [n_fsize] bytes, > 0, strictly ascending */
    const double *feff;          /* [3][n_fsize] efficiency in (0, 1] for HAP_INTRA / HAP_INTER / HAP_CROSS links */
} hap_profile;

/* hap_search_opts.flags */
#define HAP_OPT_NO_MAPTAB 1   /* keep no table of decoded mappings on the device: the DP kernel unranks each mapping itself */
#define HAP_OPT_NO_TRIE 16    /* keep no prefix tree of the mappings: every pass runs one warp per candidate (the tree form
                                 shares the DP rows of common stage prefixes between all mappings of a configuration) */
#define HAP_OPT_NO_FUSE 32    /* passes that walk the prefix trees let every block compute the layer times of its configuration itself
                                 (Eq. 2) instead of reading an array that a layer-cost launch wrote before; this flag keeps the
                                 separate launch (identical results) */
#define HAP_OPT_COUNT_SPLITS 64 /* instrumentation: hap_pipeline_dp passes of this problem also count the splits (k, j) their kernels
                                 evaluate, after all early exits, for hap_get_timings; costs a few percent of the pass */
#define HAP_OPT_HETERO_DISPATCH 128 /* Pruning 3 (Sec. 3.5 (3)) also counts, for every stage whose devices are of more than one
                                  type (its expert-parallel groups leave a homogeneous sub-cluster), the dispatch and combine
                                  traffic of the stage's MoE layers on the cross-type link: the number of MoE layers of the
                                  stage x the largest HAP_KXD among the stage's types is added to the cross-type transfer
                                  time the rule compares with eta x the mean stage time.  Stage times are not changed. */
#define HAP_OPT_UNIFORM 8     /* ablation "non-uniform partitioning disabled" (Sec. 5.5): every stage takes floor(N/PP) or
                                 ceil(N/PP) layers; the load-balance window is ignored */
#define HAP_OPT_EXACT 4       /* like HAP_OPT_REFINE, but the limit on the stage cost is then swept upward from the bottleneck over
                                 the stage costs, which yields the partition that minimises sum_i c_i + (M-1) max_i c_i (Eq. 4's
                                 pipeline term in closed form) over ALL partitions of the candidate; integer mode only.  The
                                 reported bottleneck stays that of the min-max recurrence. */
#define HAP_OPT_REFINE 2      /* after the min-max recurrence, choose among the bottleneck-optimal partitions the one with
                                 the smallest sum of stage costs (Eq. 4's T_edge), smallest split on ties; integer mode only.
                                 Costs, partitions, levels and the plan then refer to that partition; the DP tables
                                 returned by hap_pipeline_dp remain those of the min-max recurrence. */

typedef struct {
    int32_t npp, ntpe;
    const int32_t *pp_list, *tpe_list;  /* pipeline and expert-TP degrees to try (ascending; pp_list without repeats) */
    int32_t tp_max;                      /* TP and TPE are limited to this */
    int32_t delta_q;                     /* load-balance window delta in 1/1024 (Pruning 1); < 0 disables */
    uint64_t map_cap;                    /* enumerate all distinct stage-type sequences only up to this count (<= 2^56) */
    int32_t n_rc;                        /* recomputation policies, 1..HAP_MAX_RC_MASKS */
    const uint32_t *rc_masks;            /* [n_rc] bit r set: level r allowed; per stage the lowest feasible allowed level is used */
    int32_t prune;                       /* hap_search_* may skip candidates whose lower bound exceeds the incumbent */
    int32_t flags;                       /* HAP_OPT_* bits */
    int32_t eta_q;                       /* Pruning 3: drop a candidate whose cross-type transfer time per micro-batch exceeds
                                            eta x its mean stage time; eta in 1/1024 (2048 = the paper's default 2); <= 0: off */
} hap_search_opts;

/* One accepted parallel configuration x micro-batch size.  Candidate index of
 * (map_idx, rc_idx) in configuration p: offset + map_idx * n_rc + rc_idx. */
typedef struct {
    int32_t PP, TP, CP, DP, EP, TPE, b, M, EDP, G;
    int32_t itp, icp, ib, iep, mode, reserved;
    uint64_t nmap, offset;
} hap_pconf;

/* Decoded candidate (device mapping {h_i} of Sec. 3.2 plus the recomputation policy). */
typedef struct {
    uint64_t index;
    uint32_t pconf, rc_mask;
    uint64_t map_idx;
    uint8_t PP, pad[7];
    uint8_t mask[HAP_MAX_PP];   /* bit h: stage overlaps device type h */
    uint8_t link[HAP_MAX_PP];   /* boundary into stage s>=1: class | sending type << 2 | receiving type << 4 */
} hap_candidate;

/* The plan of Sec. 3.2 "Output": configuration, partition, device mapping, recomputation. */
typedef struct {
    uint64_t index;
    int32_t PP, TP, CP, DP, EP, TPE, b, M;
    uint32_t rc_mask, pad;
    uint8_t n[HAP_MAX_PP];      /* layers per stage, sum = N */
    uint8_t mask[HAP_MAX_PP];   /* device types of each stage */
    uint8_t r[HAP_MAX_PP];      /* recomputation level per stage */
    int64_t T_iter, bottleneck, T_pipe, T_sync, T_opt;
} hap_plan;

typedef struct {
    uint64_t n_pconf, n_candidates;
    uint64_t n_evaluated;   /* candidates whose dynamic program ran */
    uint64_t n_pruned;      /* candidates skipped by the lower bound */
    uint64_t n_feasible;    /* evaluated candidates with a finite cost */
    float ms_layer_cost, ms_dp, ms_total;   /* CUDA-event times of the phases on `stream` */
} hap_search_stats;

typedef struct hap_problem hap_problem;

/* Sec. 3.2: takes the planner's inputs.  Validates, copies the descriptors and uploads the
 * tables to the current device.  *out is NULL on failure. */
hap_status hap_problem_create(const hap_model *, const hap_cluster *, const hap_profile *,
                              const hap_search_opts *, hap_problem **out);
/* Waits for the problem's device work and releases it.  Its device memory is not returned to the driver but kept
 * (up to 24 blocks and 4 GiB per process) for the next hap_problem_create / hap_enumerate of the same device, which
 * reuse a block that fits with at most a quarter to spare: allocating and freeing a problem's arenas costs about as
 * much as a whole search.  No counterpart in the paper (resource management of this library). */
void hap_problem_destroy(hap_problem *);
/* Returns every idle block of that cache, on every device, to the driver (cudaFree).  Blocks of live problems are
 * not touched.  HAP_E_CUDA if a free failed. */
hap_status hap_release_cached_memory(void);

/* Sec. 3.5 / 5.1 "searches the 6D parallel space": enumerates every (PP,TP,CP,DP,EP,TPE) with
 * PP*TP*CP*DP = #devices, EP*TPE | TP*CP*DP, EP | E, x micro-batch size, in a fixed
 * lexicographic order, counts the stage mappings of each and builds the device-side tables.
 * What depends on the model's dimensions, the cluster and the search options only -- the configuration table, the
 * work items and the prefix trees of the classes' stage mappings -- is kept per process (host memory, at most a few
 * hundred entries, keyed by exactly those inputs) and reused when a later problem has the same key: planning again on
 * the same cluster with new profiled tables skips the loop nest and the tree build.  The device copies are still the
 * problem's own; the table and the address-free part of the trees are uploaded straight from page-locked images of
 * them (one per key, the tree images at most 16 per process). */
hap_status hap_enumerate(hap_problem *, uint64_t *n_pconf, uint64_t *n_candidates);
hap_status hap_get_pconfs(const hap_problem *, hap_pconf *host_out, uint64_t cap);

/* Device assignment {h_i}: decodes candidates [first, first+count) into dev_out[count]. */
hap_status hap_decode(hap_problem *, uint64_t first, uint64_t count, hap_candidate *dev_out, void *stream);

/* Eq. 2, Eq. 3, load-imbalance scaling, exposed collective time, memory model coefficients
 * (Sec. 3.3), T_dp-sync / T_opt coefficients (Eq. 4).
 * dev_c2:   [n_pconf][n_types][N][2] forward/backward ns per layer (nullable)
 * dev_coef: [n_pconf][n_types][HAP_NCOEF] (nullable)
 * hap_eval_layer_costs_f64 writes the unrounded fp64 values in the same layouts. */
hap_status hap_eval_layer_costs(hap_problem *, int64_t *dev_c2, int64_t *dev_coef, void *stream);
hap_status hap_eval_layer_costs_f64(hap_problem *, double *dev_c2, double *dev_coef, void *stream);

/* Sec. 3.5 (non-uniform layer assignment, Pruning 1 and 2) with the min-max recurrence
 * DP[i][j] = min_k max(DP[i-1][k], cost_i(k,j)), backtrace, and Eq. 4 in the closed form
 * sum_i c_i + (M-1) max_i c_i + T_dp-sync + T_opt, for candidates [first, first+count).
 * The layer costs (Eq. 2) are recomputed first: inside the blocks of the dynamic program where the pass walks the
 * classes' prefix trees (the default), into library-owned memory by a separate launch otherwise.  No candidate is
 * skipped.
 * dev_cost, dev_bottleneck: [count] (HAP_INF when infeasible)
 * dev_partition, dev_recompute: [count][HAP_MAX_PP] (nullable; zero when infeasible)
 * dev_dp_table: [count][HAP_MAX_PP+1][N+1] int64, rows 0..PP written (nullable)
 * dev_choice:   [count][HAP_MAX_PP+1][N+1] uint8, smallest optimal split k, 255 = none (nullable) */
hap_status hap_pipeline_dp(hap_problem *, uint64_t first, uint64_t count, int64_t *dev_cost,
                           int64_t *dev_bottleneck, uint8_t *dev_partition, uint8_t *dev_recompute,
                           int64_t *dev_dp_table, uint8_t *dev_choice, void *stream);

/* fp64 mode of hap_pipeline_dp: layer times and time coefficients stay unrounded doubles (the recomputation
 * factor is tau_q / 1024.0, an infeasible cost is +infinity); the memory test uses the same integer byte
 * coefficients as the integer mode.  Results agree with a plain fp64 evaluation to about 1e-12 relative
 * (prefix sums are formed in a different order), not bit for bit.
 * dev_cost, dev_bottleneck: [count] double; dev_partition, dev_recompute: [count][HAP_MAX_PP] (nullable). */
hap_status hap_pipeline_dp_f64(hap_problem *, uint64_t first, uint64_t count, double *dev_cost,
                               double *dev_bottleneck, uint8_t *dev_partition, uint8_t *dev_recompute,
                               void *stream);
/* fp64 mode of hap_search_range (no pruning).  The plan's time fields are the fp64 values rounded to
 * integer ns; the unrounded iteration time and bottleneck go to host_T_iter / host_bottleneck (nullable).
 * Synchronises `stream`. */
hap_status hap_search_range_f64(hap_problem *, uint64_t first, uint64_t count, hap_plan *host_out,
                                double *host_T_iter, double *host_bottleneck, void *stream);

/* Eq. 1: layer costs, dynamic program and argmin over candidates [first, first+count) with
 * ties going to the lowest index; writes the plan to host memory.  Synchronises `stream`.
 * host_stats is nullable.  Returns HAP_E_INFEASIBLE when no candidate is feasible.
 * With opts.prune, blocks whose configuration-level lower bound exceeds the incumbent are skipped (strict bound:
 * same plan).  Under HAP_OPT_REFINE / HAP_OPT_EXACT a plain pass first bounds every candidate from below by
 * S + (M-1) B* (B* its bottleneck, S the configuration's sum over layers of the cheapest type's time) and the
 * refinement runs only for candidates whose bound does not exceed the incumbent; host_stats->n_pruned counts the
 * candidates cut this way, candidates without a feasible partition count as evaluated.  The first such call
 * allocates 8 bytes per candidate of scratch.
 * The plan (partition, levels, terms of Eq. 4) comes from the search itself when every class walks its prefix tree:
 * each block leaves the plan of its best candidate and the winner's is copied out (the first search of a problem
 * allocates 112 bytes per block for them); otherwise the winner is evaluated once more alone. */
hap_status hap_search_range(hap_problem *, uint64_t first, uint64_t count, hap_plan *host_out,
                            hap_search_stats *host_stats, void *stream);
/* The whole candidate space. */
hap_status hap_search_best(hap_problem *, hap_plan *host_out, hap_search_stats *host_stats, void *stream);

/* Lexicographic (cost, index) minimum of a device cost array: writes dev_out[0] = cost,
 * dev_out[1] = index (as int64) of the minimum of dev_cost[0..count). */
hap_status hap_argmin(hap_problem *, const int64_t *dev_cost, uint64_t count, int64_t *dev_out, void *stream);

/* No counterpart in the paper: a variant of hap_argmin for callers that must not allocate.
 *
 * Some users of this library run it inside a process whose device memory has already been handed
 * over in full to another owner (a framework's caching allocator, a fixed arena sized at start-up),
 * or inside a steady-state loop where cudaMalloc / cudaFree are unwelcome because they can fail once
 * memory is committed and because they stall the whole device.  Such a caller cannot create a
 * hap_problem (that allocates) just to reduce a cost array it already holds.  This entry point needs
 * no problem handle and calls no cudaMalloc, cudaFree or other allocating routine: the per-block
 * partial minima go to a 64 KiB array that is part of the library image, so every GPU that loads the
 * library keeps those 64 KiB until the process exits.
 *
 * dev_cost: [count] int64 on the current device; dev_out: 2 x int64 on the same device, receives
 * (minimum cost, its lowest index).  Kernels are enqueued on `stream`; the call does not wait.
 * Limit: 1 <= count <= HAP_ARGMIN_STATIC_MAX_COUNT, otherwise HAP_E_RANGE and nothing is launched.
 * The first call on a device looks up the array's device address (one runtime query, cached per
 * device); make that first call outside any stream capture.  All calls on a device share the one
 * array and it keeps whatever the last call left there; a call writes every partial it later reads,
 * so nothing needs clearing, but two calls whose kernels overlap on the GPU (different streams)
 * race on it: keep calls on one device ordered. */
#define HAP_ARGMIN_STATIC_MAX_COUNT ((uint64_t)1 << 26)
hap_status hap_argmin_static(const int64_t *dev_cost, uint64_t count, int64_t *dev_out, void *stream);

/* Sec. 3.5 / Algorithm 1 (HS-DP over the device-group state), with the min-max objective of this library: for every
 * configuration whose stages are homogeneous (the per-stage device count divides every type's device count) and
 * every recomputation policy, the minimum over ALL stage-type sequences -- not only the enumerated mappings -- of
 * the pipeline bottleneck, from one recurrence over (layers placed, stages of each type used, type of the last
 * stage).  dev_out: [n_pconf][n_rc] int64; HAP_INF when no sequence is feasible, -1 for configurations whose
 * stages are not homogeneous.  Recomputes the layer costs into library-owned memory first; the first call
 * allocates its state tables and scratch.  Asynchronous on `stream`. */
hap_status hap_joint_bottleneck(hap_problem *, int64_t *dev_out, void *stream);

/* Measurement aid: the number of recurrence cells (i, j, k) of candidates [first, first+count) whose stage
 * cost is finite, i.e. k inside the load-balance window of stage i (Pruning 1) and the span within the memory
 * limit at some allowed recomputation level (Pruning 2).  This is the recurrence work the method defines for
 * the range, independent of what the dynamic-program kernel skips or shares.  Synchronises `stream`. */
hap_status hap_count_cells(hap_problem *, uint64_t first, uint64_t count, uint64_t *host_cells, void *stream);

/* Measurement aid: CUDA-event durations (ms) of the layer-cost kernel and of the dynamic-program
 * kernel of the most recent hap_pipeline_dp / hap_search_* call, and -- for a problem created with
 * HAP_OPT_COUNT_SPLITS, 0 otherwise -- the number of splits (k, j pairs inside the window and the memory limit) that
 * a hap_pipeline_dp launch evaluated, counted after its early exits: the work executed, as opposed to
 * hap_count_cells, the work the recurrence defines.  ms_layer_cost covers what precedes the
 * dynamic program in the pass (the per-type constants and stage coefficients, and the layer-cost launch when the
 * pass has one).  Waits for that call's kernels.  Any output may be NULL. */
hap_status hap_get_timings(hap_problem *, float *ms_layer_cost, float *ms_dp, uint64_t *cells);

/* Appendix B: the iteration latency of GIVEN plans with the steady-state term written through the index s_max of
 * the (first) bottleneck stage, T_iter = T_edge + T_middle + T_dp-sync + T_opt with T_edge = sum_i (t_f,i + t_b,i)
 * (Eq. 4) and T_middle = sum_{i <= s_max} t_f,i + (M - s_max - 1) max_i (t_f,i + t_b,i), stages 1-based, the
 * multiplier taken as 0 when negative.  t_f,i: forward time of the stage's layers (slowest member type per layer);
 * t_b,i: the rest of the stage cost (backward time, recomputation at the stage's level, stage constant), so that
 * t_f,i + t_b,i is the stage cost of the recurrence.  A post-hoc evaluator: it does not choose partitions.
 * Candidates [first, first+count); dev_partition / dev_recompute: [count][HAP_MAX_PP] layers and levels per stage
 * as hap_pipeline_dp wrote them for the same range; dev_t_iter: [count] out, HAP_INF where the layer counts do
 * not partition the N layers (an infeasible candidate); dev_detail: [count][3] out, T_edge, T_middle, s_max
 * (nullable).  Recomputes the layer costs into library-owned memory first.  Asynchronous on `stream`. */
hap_status hap_eval_appendix_b(hap_problem *, uint64_t first, uint64_t count, const uint8_t *dev_partition,
                               const uint8_t *dev_recompute, int64_t *dev_t_iter, int64_t *dev_detail, void *stream);

/* Sec. 3.3 names the 1F1B schedule; Eq. 4 and Appendix B put its iteration latency in closed form.  This entry
 * point runs the schedule itself for GIVEN plans, to measure what the closed forms leave out on unequal stages:
 * stage i of PP runs min(PP - i, M) warm-up forward passes, then forward / backward pairs while forwards remain,
 * then the remaining backward passes; F(i, m) starts when the stage is free and F(i-1, m) has ended, B(i, m) when
 * the stage is free and B(i+1, m) has ended (last stage: its own F(i, m)); a forward pass of stage i takes t_f,i,
 * a backward pass t_b,i (the split of hap_eval_appendix_b, so transfers are part of the passes).
 * Candidates [first, first+count); dev_partition / dev_recompute: [count][HAP_MAX_PP] as hap_pipeline_dp wrote
 * them for the same range; dev_t_iter: [count] out, time the last backward pass ends + T_sync + T_opt, HAP_INF
 * where the layer counts do not partition the N layers; dev_detail: [count][2] out, the simulated pipeline time
 * and Eq. 4's pipeline term sum_i c_i + (M-1) max_i c_i of the same plan (nullable).  A post-hoc evaluator: one
 * warp per plan and about 2 (M + PP) rounds each, meant for chosen plans, not for the whole candidate space.
 * Recomputes the layer costs into library-owned memory first.  Asynchronous on `stream`. */
hap_status hap_simulate_1f1b(hap_problem *, uint64_t first, uint64_t count, const uint8_t *dev_partition,
                             const uint8_t *dev_recompute, int64_t *dev_t_iter, int64_t *dev_detail, void *stream);

/* Sec. 4 caches the profiled tables between planner runs; these two calls do that for a whole planning problem.
 * hap_problem_save writes everything hap_problem_create was given (model, cluster, tables, coefficients, search
 * options; the tables are read back from the device) as one self-describing blob into host_buf and sets *host_need
 * to its size; with host_buf = NULL it only reports the size, with cap < size it writes nothing and returns
 * HAP_E_RANGE.  hap_problem_load validates a blob (magic, length, every array length) and hands its content to
 * hap_problem_create on the current device; a blob that is truncated, altered in size or of another version gives
 * HAP_E_INVALID.  The blob is host-endian and tied to this header's limits; it carries no results. */
hap_status hap_problem_save(hap_problem *, void *host_buf, uint64_t cap, uint64_t *host_need);
hap_status hap_problem_load(const void *host_buf, uint64_t len, hap_problem **out);
/* Layers, device types and recomputation policies of a problem (what a caller needs to size the outputs of a loaded
 * problem); any pointer may be NULL. */
hap_status hap_problem_dims(const hap_problem *, int32_t *host_N, int32_t *host_T, int32_t *host_n_rc);

/* Self-checking build (no counterpart in the paper).  A library compiled with -DHAP_CHECKED
 * (paper_2609_39350_b200.build.build_library(checked=True) -> libhap_checked.so) compares the indices and
 * shared-memory addresses its kernels form from tables (tree records, row origins, threshold indices, output slots,
 * ring slots of the schedule simulation) with their bounds before use; a violation sets a bit per check site in a
 * device word and skips the access, so nothing faults.  hap_self_check waits for the current device, returns the
 * sites that fired since the last call in *host_sites (0: none) and clears the word.  In the normal build the checks
 * are compiled away and the call returns HAP_E_STATE with *host_sites = 0. */
hap_status hap_self_check(uint64_t *host_sites);

/* Measurement aid: the number of kernels one hap_pipeline_dp call over the whole candidate space followed by
 * one hap_argmin call launches (the two layer-cost kernels, the candidate decode and the tree gather - one launch
 * each for all PP classes when every class walks its prefix tree, else per class -, the dynamic program per PP
 * class, the two reduction kernels).  Host value, no device work. */
hap_status hap_launches_per_pass(hap_problem *, uint32_t *host_count);

const char *hap_status_str(hap_status);
const char *hap_last_error(const hap_problem *);

#ifdef __cplusplus
}
#endif
#endif /* HAP_H */

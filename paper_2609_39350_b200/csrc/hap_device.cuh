// Device-side data layout and kernels of libhap (sm_100a).
//
// Kernels
//   type_const_kernel   per (configuration, type): constants of Eq. 2 / Eq. 3 and the 21 stage
//                       coefficients, fp64 with one IEEE operation per operator (the translation
//                       unit is compiled with --fmad=false), three independent roles per pair.
//   layer_cost_kernel   per (configuration, type, layer): Eq. 2 with imbalance scaling, rounding,
//                       one block per configuration, one thread per layer.
//   decode_kernel       candidate index -> stage type masks and boundary link classes;
//   maptab_kernel       the same for every mapping of one PP class; maptab_all_kernel for all classes in one
//                       launch (every pass).
//   trie_dp_kernel      (hap_trie.cuh) the default dynamic program: all mappings of a configuration
//                       together through the prefix tree of their stage sequences.
//   pipeline_dp_kernel  the general form (DP tables on request, refinement / exact modes, classes
//                       without a tree): one warp per candidate, stage rows and memory-threshold tables in shared
//                       memory (built once per block for the block's configuration), min-max
//                       recurrence with lanes over the end layer j, optional refinement pass,
//                       backtrace, Eq. 4 closed form, Pruning 3; in search mode the block-level
//                       (cost, index) minimum and lower-bound pruning against an atomic incumbent.
//                       Instantiated on int64 (exact) and double (fp64 mode).
//   joint_dp_kernel     recurrence over the device-group state: minimum bottleneck over all
//                       stage-type sequences of a configuration.
//   appendix_b_kernel   iteration latency of given plans by the appendix's steady-state expression.
//   simulate_1f1b_kernel  iteration latency of given plans by an event simulation of the 1F1B schedule.
//   argmin kernels      lexicographic (cost, index) minimum, block partials then one block.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include "../../include/hap.h"

namespace hap {

typedef long long i64;
typedef unsigned long long u64;
typedef unsigned int u32;

// Self-checking build (-DHAP_CHECKED): what a memory checker would do from outside, done by the kernels themselves.
// Indices and shared-memory addresses that a kernel forms from tables (tree records, row origins, threshold
// indices, output slots) are compared with their bounds before use; a violation sets the site's bit in a device
// word and the access is skipped: nothing traps, the launch completes, hap_self_check() returns the word.
// The normal build compiles every check away.
//   site 0 shared-memory address outside the block's allocation or misaligned    1 row-buffer slot
//        2 split-choice slot    3 output slot    4 tree node    5 split index read back    6 threshold index
//        7 configuration index  8 decoded-mapping table    9 ring slot of the schedule simulation
#ifdef HAP_CHECKED
__device__ unsigned long long g_hap_check_sites;
#define HAP_CHECK_OK(site, cond) ((cond) ? true : (atomicOr(&hap::g_hap_check_sites, 1ull << (site)), false))
#else
#define HAP_CHECK_OK(site, cond) (true)
#endif

constexpr int kMaxMasks = (1 << HAP_MAX_TYPES) - 1;
constexpr int kDpWarps = 12;          // most warps per block of the DP kernel
constexpr i64 kInf = (i64)1 << 62;

// Everything a kernel needs besides the big tables; passed by value.
struct DevConst {
    int N, T, R, n_rc, ntp, ncp, nmb, nep;
    int S, H, E, k, n_shared, F_dense, F_exp, nq, nkv, V, GB;
    int delta_q, tau_linear, eta_q, uniform;
    int het_dispatch;                 // Pruning 3 also counts the dispatch / combine traffic of stages that span device types
    int kind_uniform;                 // every layer is of one kind (all MoE or all dense): a span's memory depends on its length only
    int kind_uniform_from;            // first layer u such that layers u..N-1 are all of one kind (0 when kind_uniform)
    double beta, kappa, chi, gamma, ovl_tp, ovl_cp, ovl_dp, capf;
    double alpha[3];
    double eta[HAP_MAX_TYPES], croute[HAP_MAX_TYPES], copt[HAP_MAX_TYPES];
    double bw_intra[HAP_MAX_TYPES], bw_inter[HAP_MAX_TYPES];
    double act_coef[2];
    double rho[HAP_MAX_LIST];
    i64 P[HAP_MAX_TYPES], cap_eff[HAP_MAX_TYPES], m[HAP_MAX_TYPES];
    int node_size[HAP_MAX_TYPES];
    int n_fsize;                      // communication-primitive table: link efficiency by message size (0: none)
    double fsize[HAP_MAX_LIST], feff[3][HAP_MAX_LIST];
    unsigned rc_masks[HAP_MAX_RC_MASKS];
    int rc_order[HAP_MAX_RC_MASKS];   // policies from the most permissive to the most restrictive
    unsigned rc_sup[HAP_MAX_RC_MASKS]; // per position in rc_order: earlier positions whose allowed levels are a superset
    int xi_q[HAP_MAX_RC], tau_q[HAP_MAX_RC];
    u64 kindbits[4];                  // bit l set: layer l is an MoE layer
    const double *tab4;               // [type][tp][cp][mb][layer] x (t_dense fwd, t_dense bwd, t_ffn fwd, t_ffn bwd), 32-byte records
    const double *tpre, *tpost;
    const hap_pconf *pconf;           // device copy of the configuration table
    u64 n_pconf;
};

// One block of DP work: mappings [lo, lo+count) of configuration p, every recompute policy.
struct WorkItem {
    uint32_t p;
    uint32_t count;
    u64 lo;
};

// What a block of a search leaves beside its (cost, index) minimum when it can: the plan of that candidate.
struct __align__(16) PlanSlot {
    i64 bott, T_pipe, T_sync, T_opt;
    uint8_t n[HAP_MAX_PP], r[HAP_MAX_PP];     // layers and recomputation level of stages 1..PP (the rest is not written)
    int PP, pad[3];
};
static_assert(HAP_MAX_PP == 32 && sizeof(PlanSlot) % 16 == 0, "the plan bytes move as 16-byte pieces");

struct DpOut {
    i64 *cost, *bottleneck;
    uint8_t *partition, *recompute;
    i64 *dp_table;
    uint8_t *choice;
    i64 *detail;                      // [count][3] T_pipe, T_sync, T_opt (nullable)
    u64 first, count;                 // global candidate range that is written
    const i64 *first_dev;             // if set: `first` is read from here by the kernel (a negative value: nothing is written)
    // search mode
    i64 *partial_cost;                // [gridDim.x]
    u64 *partial_index;               // [gridDim.x]
    u64 *counters;                    // [0] evaluated, [1] feasible, [2] pruned, [4] recurrence cells (nullable)
    u64 *incumbent;                   // running minimum of T_iter, for pruning
    const i64 *lb_sum;                // per configuration: sum over layers of the cheapest type's time
    int prune;                        // search mode: skip blocks whose lower bound exceeds the incumbent
    int exact;                        // refinement kernels: sweep the stage-cost limit for the optimum of sum + (M-1) max
    int count_only;                   // instrumentation: count the finite-cost cells of each candidate, run no recurrence
    // layer costs computed by the DP blocks themselves (prefix-tree kernel): per (configuration, type) constants of
    // Eq. 2; null: the blocks read the layer-cost array.  range_flag: set when a layer time leaves the supported range
    const struct TypeConst *tcg;
    u64 *range_flag;
    // search with the refinement / exact objective: per-candidate lower bounds on T_iter from a preceding plain pass,
    // indexed by the global candidate index (HAP_INF: the candidate has no feasible partition); a candidate whose
    // bound exceeds the incumbent is skipped
    const i64 *cand_lb;
    PlanSlot *block_plan;             // search over the prefix trees: per block the plan of its best candidate (nullable)
    int force_plain;                  // run the plain min-max pass although the problem asks for a refinement mode
};

// ------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ int moe_before(const DevConst &dc, int l)
{   // number of MoE layers among layers 0..l-1
    int n = 0;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        int lo = w * 64;
        if (l >= lo + 64) n += __popcll(dc.kindbits[w]);
        else if (l > lo) n += __popcll(dc.kindbits[w] & ((1ull << (l - lo)) - 1ull));
    }
    return n;
}

__device__ __forceinline__ int layer_kind(const DevConst &dc, int l)
{
    return (int)((dc.kindbits[l >> 6] >> (l & 63)) & 1ull);
}

__device__ __forceinline__ i64 shfl_i64(i64 v, int src)
{
    return __shfl_sync(0xffffffffu, v, src);
}

__device__ __forceinline__ i64 warp_max_i64(i64 v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) { i64 t = __shfl_xor_sync(0xffffffffu, v, o); v = t > v ? t : v; }
    return v;
}

__device__ __forceinline__ i64 warp_sum_i64(i64 v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// lexicographic minimum of (cost, index) over the warp
__device__ __forceinline__ void warp_argmin(i64 &c, u64 &ix)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        i64 c2 = __shfl_xor_sync(0xffffffffu, c, o);
        u64 i2 = __shfl_xor_sync(0xffffffffu, ix, o);
        if (c2 < c || (c2 == c && i2 < ix)) { c = c2; ix = i2; }
    }
}

// ------------------------------------------------------------------------------------------
// layer cost (Eq. 2, Eq. 3) and stage coefficients
// ------------------------------------------------------------------------------------------
struct LinkCtx { double bw_intra, bw_inter; int node_size; };

__device__ __forceinline__ int link_class(const LinkCtx &lc, i64 ext) { return ext <= lc.node_size ? HAP_INTRA : HAP_INTER; }
__device__ __forceinline__ double link_bw(const LinkCtx &lc, int cls) { return cls == HAP_INTRA ? lc.bw_intra : lc.bw_inter; }

// Volume term of a communication primitive (the communication-primitive table of Sec. 3.4): vol bytes over a link
// of class cls with nominal bandwidth bw take vol / bw divided by the link's profiled efficiency at that message
// size, piecewise linear between the profiled sizes and constant outside them; no table: efficiency 1.
__device__ __forceinline__ double link_eff(const DevConst &dc, int cls, double vol)
{
    const int n = dc.n_fsize;
    if (vol <= dc.fsize[0]) return dc.feff[cls][0];
    if (vol >= dc.fsize[n - 1]) return dc.feff[cls][n - 1];
    int i = 0;
    while (vol >= dc.fsize[i + 1]) ++i;
    return dc.feff[cls][i] + (vol - dc.fsize[i]) * ((dc.feff[cls][i + 1] - dc.feff[cls][i]) / (dc.fsize[i + 1] - dc.fsize[i]));
}

__device__ __forceinline__ double xfer_ns(const DevConst &dc, int cls, double vol, double bw)
{
    const double t = vol / bw;
    if (dc.n_fsize <= 0) return t;
    return t / link_eff(dc, cls, vol);
}

// collective over w ranks that span `ext` consecutive devices, D bytes per rank
__device__ __forceinline__ double collective_ns(const DevConst &dc, const LinkCtx &lc, i64 w, i64 ext, double D)
{
    if (w == 1) return 0.0;
    const int cls = link_class(lc, ext);
    const double lat = dc.alpha[cls] * (double)(w - 1);
    const double vol = (D * (double)(w - 1)) / (double)w;
    return lat + xfer_ns(dc, cls, vol, link_bw(lc, cls));
}

struct __align__(16) TypeConst {      // per (configuration, type) values used by every layer, in the pairs the layer kernel reads
    double den, rden;               // expert-term divisor (Eq. 3) and its correctly rounded reciprocal
    double disp2, imb;              // twice the dispatch time, load-imbalance factor
    double tr, tr2;                 // router term, forward and backward
    double commF_moe, commB_moe;    // exposed collective time of an MoE layer, forward and backward
    double commF_dense, commB_dense;
    long long row, pad;             // table row (itp, icp, ib) of the configuration
};

template <bool QUANT>
__device__ __forceinline__ void store_pair(i64 *qi, double *qd, size_t at, double a, double b)
{
    if (QUANT) {
        longlong2 v; v.x = __double2ll_rn(a); v.y = __double2ll_rn(b);
        *reinterpret_cast<longlong2 *>(qi + at) = v;
    } else {
        double2 v; v.x = a; v.y = b;
        *reinterpret_cast<double2 *>(qd + at) = v;
    }
}

constexpr int kLcThreads = 128;

// Eq. 2 for one (configuration, device type, layer): forward and backward time of the layer from its table entries
// ta = (t_dense fwd, bwd), tf = (t_ffn fwd, bwd) and the per-(configuration, type) constants tc (a TypeConst read as
// 16-byte pairs).  One IEEE operation per operator, in the order the formulas are written.
__device__ __forceinline__ double div_by(double a, double b, double y);
__device__ __forceinline__ u64 find_pconf(const DevConst &dc, u64 c);
__device__ __forceinline__ void layer_cost_pair(const double2 *tc, double2 ta, double2 tf, bool dense, double kappa, double &cf, double &cb)
{
    if (dense) {
        const double2 cm = tc[4];                                // commF_dense, commB_dense
        cf = ta.x + cm.x;
        cb = ta.y + cm.y;
    } else {
        const double2 dn = tc[0], di = tc[1], tr = tc[2], cm = tc[3];
        const double xf = div_by(kappa * tf.x, dn.x, dn.y);
        const double mf = (xf + di.x) * di.y;
        cf = (((ta.x - tf.x) + mf) + tr.x) + cm.x;
        const double xb = div_by(kappa * tf.y, dn.x, dn.y);
        const double mb = (xb + di.x) * di.y;
        cb = (((ta.y - tf.y) + mb) + tr.y) + cm.y;
    }
}

// a / b for a divisor whose correctly rounded reciprocal y = RN(1/b) is known: q0 = RN(a*y), the exact
// residual r = a - b*q0 (one fused operation) and q = RN(q0 + r*y) give the correctly rounded quotient
// (Markstein's division theorem), i.e. the same bits as the IEEE division a / b, at three operations.
__device__ __forceinline__ double div_by(double a, double b, double y)
{
    const double q0 = a * y;
    const double r = __fma_rn(-b, q0, a);
    return __fma_rn(r, y, q0);
}

// Phase 1 (type_const_kernel): per (configuration, type) the constants of Eq. 2 / Eq. 3 (into a scratch array)
// and the 21 stage coefficients.  The work of one (configuration, type) is a chain of about 40 fp64 divisions,
// so it is cut into three independent roles (blockIdx.y: layer constants; p2p / activation / extra-memory
// coefficients; weight / sync / optimizer coefficients), one thread per (configuration, type) and role.
// Phase 2 (layer_cost_kernel): one block per configuration, one thread per layer.
template <bool QUANT>
__device__ __forceinline__ bool put_coef(i64 *coef, double *coeff, size_t at, int q, double v)
{
    if (QUANT) coef[at + q] = __double2ll_rn(v);
    else coeff[at + q] = v;
    // time coefficients must stay below 2^40 ns (per-layer ones below 2^36), bytes below 2^50
    const double lim = (q <= HAP_SLAT || q == HAP_KXD) ? 1.0995e12 : (q < HAP_MW ? 6.8719e10 : 1.1259e15);
    return !(v < lim);
}

template <bool QUANT>
__global__ void __launch_bounds__(kLcThreads)
type_const_kernel(const DevConst dc, TypeConst *tcg, i64 *coef, double *coeff, u64 *range_flag, unsigned p_first, unsigned n_conf)
{
    // the layer-cost kernel behind this one may start its table reads now (programmatic dependent launch)
    asm volatile("griddepcontrol.launch_dependents;");
    const int T = dc.T;
    const int role = blockIdx.y;
    const i64 H = dc.H;
    const u64 gid = (u64)blockIdx.x * kLcThreads + threadIdx.x;
    const u64 p = (u64)p_first + gid / HAP_MAX_TYPES;          // configurations [p_first, p_first + n_conf)
    const int h = (int)(gid % HAP_MAX_TYPES);
    if (gid / HAP_MAX_TYPES >= n_conf || p >= dc.n_pconf || h >= T) return;
    const bool want_coef = (QUANT && coef) || (!QUANT && coeff);
    if (role != 0 && !want_coef) return;
    const hap_pconf pc = dc.pconf[p];
    const int TP = pc.TP, CP = pc.CP, DP = pc.DP, EP = pc.EP, TPE = pc.TPE, EDP = pc.EDP, b = pc.b;
    const i64 G = pc.G;
    const i64 tok = (i64)((unsigned)b * (unsigned)dc.S / (unsigned)CP);
    const i64 Hkv = (i64)((unsigned)dc.H * (unsigned)dc.nkv / (unsigned)dc.nq);
    const double thb = (double)tok * (double)H;
    const double Dtp = thb * dc.beta;
    LinkCtx lc; lc.bw_intra = dc.bw_intra[h]; lc.bw_inter = dc.bw_inter[h]; lc.node_size = dc.node_size[h];
    const size_t at = ((size_t)p * T + h) * HAP_NCOEF;
    bool bad = false;

    if (role == 0) {
        TypeConst tc;
        tc.imb = 1.0 + dc.gamma * (dc.rho[pc.iep] - 1.0);
        double tdisp = 0.0;
        if (EP != 1) {
            const double Dmoe = ((thb * dc.beta) * (double)dc.k) * (1.0 - 1.0 / (double)EP);
            const double Dag = (thb * dc.beta) * (double)(EP - 1);
            const int cls = link_class(lc, (i64)EP * TPE);
            const double fa = dc.alpha[cls] * (double)(EP - 1) + xfer_ns(dc, cls, Dmoe, link_bw(lc, cls));
            const double fg = dc.alpha[cls] * (double)(EP - 1) + xfer_ns(dc, cls, Dag, link_bw(lc, cls));
            tdisp = (fa <= fg) ? fa : fg;
        }
        tc.disp2 = 2.0 * tdisp;
        const double ttpA = 2.0 * collective_ns(dc, lc, TP, TP, Dtp);
        const double ttpD = ttpA;
        const double ttpM = 2.0 * collective_ns(dc, lc, TPE, TPE, Dtp);
        const double Dkv = ((((2.0 * (double)b) * (double)dc.S) * (double)Hkv) * dc.beta) / (double)TP;
        const double tcp = collective_ns(dc, lc, CP, (i64)TP * CP, Dkv);
        tc.tr = dc.croute[h] * thb;
        tc.tr2 = 2.0 * tc.tr;
        tc.commF_dense = dc.ovl_tp * (ttpA + ttpD) + dc.ovl_cp * tcp;
        tc.commB_dense = dc.ovl_tp * (ttpA + ttpD) + dc.ovl_cp * (2.0 * tcp);
        tc.commF_moe = dc.ovl_tp * (ttpA + ttpM) + dc.ovl_cp * tcp;
        tc.commB_moe = dc.ovl_tp * (ttpA + ttpM) + dc.ovl_cp * (2.0 * tcp);
        tc.den = (dc.eta[h] * (double)EP) * (double)TPE;
        tc.rden = 1.0 / tc.den;
        tc.row = (pc.itp * dc.ncp + pc.icp) * dc.nmb + pc.ib;
        tc.pad = 0;
        tcg[p * T + h] = tc;
    } else if (role == 1) {
        const size_t i4 = (((size_t)h * dc.ntp + pc.itp) * dc.ncp + pc.icp) * dc.nmb + pc.ib;
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_KPRE, dc.tpre[i4]);
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_KPOST, dc.tpost[i4]);
        const double Dp = Dtp / (double)TP;
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_KP2P_INTRA, 2.0 * (dc.alpha[HAP_INTRA] + xfer_ns(dc, HAP_INTRA, Dp, dc.bw_intra[h])));
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_KP2P_INTER, 2.0 * (dc.alpha[HAP_INTER] + xfer_ns(dc, HAP_INTER, Dp, dc.bw_inter[h])));
#pragma unroll
        for (int h2 = 0; h2 < HAP_MAX_TYPES; ++h2) {
            const double bo = h2 < T ? dc.bw_inter[h2] : dc.bw_inter[h];
            const double bmin = dc.bw_inter[h] < bo ? dc.bw_inter[h] : bo;
            bad |= put_coef<QUANT>(coef, coeff, at, HAP_KP2P_CROSS + h2, 2.0 * (dc.alpha[HAP_CROSS] + xfer_ns(dc, HAP_CROSS, Dp, bmin * dc.chi)));
        }
        const i64 wd = (i64)DP * CP;
        const double shd = 6.0 + 12.0 / (double)wd;
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MA + HAP_DENSE, (thb * dc.act_coef[HAP_DENSE]) / (double)TP);
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MA + HAP_MOE, (thb * dc.act_coef[HAP_MOE]) / (double)TP);
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MX,
                               ((2.0 * ((thb * dc.beta) * (double)dc.k)) * (1.0 - 1.0 / (double)EP)) * dc.capf
                               + ((double)tok * (double)dc.E) * 4.0);
        const double mpre = (((double)dc.V * (double)H) / (double)TP) * shd;
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MPRE, mpre);
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MPOST, mpre);
        // dispatch + combine of one MoE layer (forward and backward, with the imbalance factor of Eq. 2) when the
        // expert-parallel group spans device types: Eq. 3's volumes over the cross-type link
        double kxd = 0.0;
        if (EP != 1) {
            const double Dmoe = ((thb * dc.beta) * (double)dc.k) * (1.0 - 1.0 / (double)EP);
            const double Dag = (thb * dc.beta) * (double)(EP - 1);
            const double bx = dc.bw_inter[h] * dc.chi;
            const double fa = dc.alpha[HAP_CROSS] * (double)(EP - 1) + xfer_ns(dc, HAP_CROSS, Dmoe, bx);
            const double fg = dc.alpha[HAP_CROSS] * (double)(EP - 1) + xfer_ns(dc, HAP_CROSS, Dag, bx);
            kxd = (4.0 * ((fa <= fg) ? fa : fg)) * (1.0 + dc.gamma * (dc.rho[pc.iep] - 1.0));
        }
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_KXD, kxd);
    } else {
        const i64 wd = (i64)DP * CP;
        const double shd = 6.0 + 12.0 / (double)wd;
        const double she = 6.0 + 12.0 / (double)EDP;
        const i64 Pattn = H * (H + 2 * Hkv) + H * H + 2 * H;
        const i64 Pffn_d = 3 * H * (i64)dc.F_dense, Pffn_e = 3 * H * (i64)dc.F_exp;
        const i64 Pe = (i64)(dc.E / EP) * Pffn_e;
        const i64 Prt = H * (i64)dc.E;
        i64 Pd[2];
        Pd[HAP_DENSE] = Pattn + Pffn_d;
        Pd[HAP_MOE] = Pattn + (i64)dc.n_shared * Pffn_e;
        const double PeT = (double)Pe / (double)TPE;
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MW + HAP_DENSE, ((double)Pd[HAP_DENSE] / (double)TP) * shd);
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_MW + HAP_MOE,
                               ((double)Pd[HAP_MOE] / (double)TP + (double)Prt) * shd + PeT * she);
        const int cG = link_class(lc, G);
        const double bwG = link_bw(lc, cG);
        const double vfd = (double)(wd - 1) / (double)wd, vfe = (double)(EDP - 1) / (double)EDP;
#pragma unroll
        for (int kd = 0; kd < 2; ++kd) {
            const i64 Pdd = Pd[kd] + (kd == HAP_MOE ? Prt : 0);
            const double Pel = kd == HAP_MOE ? PeT : 0.0;
            bad |= put_coef<QUANT>(coef, coeff, at, HAP_SBW + kd,
                                   dc.ovl_dp * (xfer_ns(dc, cG, (6.0 * ((double)Pdd / (double)TP)) * vfd, bwG) + xfer_ns(dc, cG, (6.0 * Pel) * vfe, bwG)));
            bad |= put_coef<QUANT>(coef, coeff, at, HAP_OPT + kd,
                                   dc.copt[h] * ((double)Pdd / (double)((i64)TP * DP * CP) + Pel / (double)EDP));
        }
        bad |= put_coef<QUANT>(coef, coeff, at, HAP_SLAT,
                               dc.ovl_dp * (dc.alpha[cG] * (2.0 * (double)(wd - 1) + 2.0 * (double)(EDP - 1))));
    }
    if (bad && range_flag) atomicOr(range_flag, 1ull);
}

// one block per configuration, one thread per layer; a thread handles its layer for every device type, so
// that up to 8 table reads of 16 bytes are in flight per thread before the first result is needed.
// KIND: 0 every layer dense, 1 every layer MoE (the branch on the layer kind is then uniform and compiled away),
// 2 mixed.  WANT_LB: also the per-configuration lower bound the search prunes with.
template <bool QUANT, int KIND, bool WANT_LB>
__global__ void __launch_bounds__(256)
layer_cost_kernel(const DevConst dc, const TypeConst *__restrict__ tcg, i64 *__restrict__ c2, double *__restrict__ c2f,
                  i64 *__restrict__ lb_sum, u64 *range_flag, const i64 *index_dev, unsigned p_first)
{
    __shared__ TypeConst tcs[HAP_MAX_TYPES];
    __shared__ i64 s_lb[8];
    const int N = dc.N, T = dc.T;
    // block b works on configuration p_first + b; or, when a preceding kernel left a candidate index in device
    // memory, on the configuration that owns it (negative: none)
    unsigned p = p_first + blockIdx.x;
    if (index_dev) {
        const i64 f = *index_dev;
        if (f < 0) return;
        p = (unsigned)find_pconf(dc, (u64)f);
    }
    const int l = threadIdx.x;
    const bool dense = KIND == 0 || (KIND == 2 && l < N && layer_kind(dc, l) == HAP_DENSE);
    double2 ta[HAP_MAX_TYPES], tf[HAP_MAX_TYPES];           // (t_dense fwd, bwd), (t_ffn fwd, bwd) of the layer per type
    if (l < N) {
        // the profiled table entries depend on the kernel's inputs only: they are requested before the wait for
        // the per-type constants of the preceding kernel
        const hap_pconf *pcf = dc.pconf + p;
        const size_t row = ((size_t)pcf->itp * dc.ncp + pcf->icp) * dc.nmb + pcf->ib;   // the same table row for every type
        const size_t stride_h = (size_t)dc.ntp * dc.ncp * dc.nmb * N * 2;                // double2 pairs between device types
        const double2 *tp = reinterpret_cast<const double2 *>(dc.tab4) + (row * N + l) * 2;
#pragma unroll
        for (int h = 0; h < HAP_MAX_TYPES; ++h) {
            if (h < T) {
                ta[h] = __ldg(tp);
                tf[h] = dense ? make_double2(0.0, 0.0) : __ldg(tp + 1);
                tp += stride_h;
            }
        }
    }
    // launched as a programmatic dependent of type_const_kernel: everything above overlaps that kernel's tail;
    // its results are visible after this wait (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    {   // stage the configuration's per-type constants (12 doubles each) in shared memory
        constexpr int W = sizeof(TypeConst) / 16;
        const double2 *src = reinterpret_cast<const double2 *>(tcg + (size_t)p * T);
        double2 *dst = reinterpret_cast<double2 *>(tcs);
        for (int q = threadIdx.x; q < T * W; q += blockDim.x) dst[q] = src[q];
    }
    __syncthreads();
    i64 lmin = 0;                       // min over device types of this layer's forward+backward time
    if (l < N) {
        bool bad = false;                                                    // a value left the supported range
        const double kappa = dc.kappa;
        i64 *o_i = c2 + ((size_t)p * T * N + l) * 2;
        double *o_d = c2f + ((size_t)p * T * N + l) * 2;
#pragma unroll
        for (int h = 0; h < HAP_MAX_TYPES; ++h) {
            if (h < T) {
                double cf, cb;
                layer_cost_pair(reinterpret_cast<const double2 *>(&tcs[h]), ta[h], tf[h], dense, kappa, cf, cb);
                bad |= !(cf < 6.8719e10) | !(cb < 6.8719e10);                 // 2^36 ns per layer
                if (QUANT) {
                    longlong2 v; v.x = __double2ll_rn(cf); v.y = __double2ll_rn(cb);
                    *reinterpret_cast<longlong2 *>(o_i) = v;
                    o_i += (size_t)N * 2;
                    if (WANT_LB) {
                        const i64 q = v.x + v.y;
                        lmin = (h == 0 || q < lmin) ? q : lmin;
                    }
                } else {
                    double2 v; v.x = cf; v.y = cb;
                    *reinterpret_cast<double2 *>(o_d) = v;
                    o_d += (size_t)N * 2;
                }
            }
        }
        if (bad && range_flag) atomicOr(range_flag, 1ull);
    }
    // every layer runs on some device type, so the sum over layers of the cheapest type's time bounds the
    // summed stage time of every candidate of this configuration from below (used by the search's pruning)
    if (QUANT && WANT_LB) {
        lmin = warp_sum_i64(lmin);
        if ((threadIdx.x & 31) == 0) s_lb[threadIdx.x >> 5] = lmin;
        __syncthreads();
        if (threadIdx.x == 0) {
            i64 t = 0;
            for (int w = 0; w < (int)(blockDim.x >> 5); ++w) t += s_lb[w];
            lb_sum[p] = t;
        }
    }
}

// ------------------------------------------------------------------------------------------
// candidate decode: every lane of the warp calls this; lane s < PP receives stage s
// ------------------------------------------------------------------------------------------
struct StageMap {
    int mask;       // types the stage overlaps
    int cls;        // link class of the boundary into the stage (stage >= 1)
    int ha, hb;     // sending / receiving device type of that boundary
};

__device__ __forceinline__ StageMap decode_stage(const DevConst &dc, const hap_pconf &pc, u64 map_idx, int lane)
{
    StageMap sm; sm.mask = 0; sm.cls = 0; sm.ha = 0; sm.hb = 0;
    const int PP = pc.PP, T = dc.T;
    const i64 G = pc.G;
    if (pc.mode == HAP_MAP_MULTISET) {
        // unrank the map_idx-th sequence (lexicographic, types ascending) of a multiset;
        // the number of completions after placing type h is tot * cnt[h] / rem (exact)
        int cnt[HAP_MAX_TYPES], used[HAP_MAX_TYPES];
#pragma unroll
        for (int h = 0; h < HAP_MAX_TYPES; ++h) { cnt[h] = h < T ? (int)(dc.m[h] / G) : 0; used[h] = 0; }
        u64 tot = pc.nmap, idx = map_idx;
        int my_h = 0, my_q = 0, prev_h = 0, last_h = 0;
        for (int pos = 0; pos < PP; ++pos) {
            const unsigned rem = (unsigned)(PP - pos);
            int pick = 0;
            bool found = false;
#pragma unroll
            for (int h = 0; h < HAP_MAX_TYPES; ++h) {
                if (!found && cnt[h] > 0) {
                    const u64 below = tot * (u64)cnt[h] / rem;
                    if (idx < below) { pick = h; tot = below; found = true; }
                    else idx -= below;
                }
            }
            int q = 0;
#pragma unroll
            for (int h = 0; h < HAP_MAX_TYPES; ++h)
                if (h == pick) { q = used[h]; used[h]++; cnt[h]--; }
            if (pos == lane) { my_h = pick; my_q = q; prev_h = last_h; }
            last_h = pick;
        }
        if (lane < PP) {
            sm.mask = 1 << my_h;
            sm.hb = my_h;
            sm.ha = prev_h;
            if (lane > 0) {
                if (prev_h != my_h) sm.cls = HAP_CROSS;
                else {
                    // consecutive stages of one type are consecutive in that type's device line
                    const i64 first = (i64)my_q * G;
                    const int ns = dc.node_size[my_h];
                    sm.cls = ((first - 1) / ns == first / ns) ? HAP_INTRA : HAP_INTER;
                }
            }
        }
    } else {
        // map_idx-th permutation of the types (lexicographic); device line = type blocks in that order
        int sigma[HAP_MAX_TYPES];
        {
            unsigned avail = (1u << T) - 1u;
            u64 idx = map_idx;
            u64 f = 1;
            for (int i = 2; i < T; ++i) f *= (u64)i;          // (T-1)!
#pragma unroll
            for (int pos = 0; pos < HAP_MAX_TYPES; ++pos) {
                sigma[pos] = 0;
                if (pos < T) {
                    int pick = (int)(idx / f);
                    idx -= (u64)pick * f;
                    if (T - 1 - pos > 0) f /= (u64)(T - 1 - pos);
                    // pick-th set bit of avail
                    unsigned a = avail;
                    for (int t = 0; t < pick; ++t) a &= a - 1;
                    const int h = __ffs(a) - 1;
                    sigma[pos] = h;
                    avail &= ~(1u << h);
                }
            }
        }
        if (lane < PP) {
            const i64 lo = (i64)lane * G, hi = lo + G - 1;
            i64 start = 0;
            int ta = 0, tb = 0;
            i64 oa = 0, ob = 0;
#pragma unroll
            for (int bq = 0; bq < HAP_MAX_TYPES; ++bq) {
                if (bq < T) {
                    const int h = sigma[bq];
                    const i64 end = start + dc.m[h];
                    if (start <= hi && end > lo) sm.mask |= 1 << h;
                    if (start <= lo && lo < end) { tb = h; ob = lo - start; }
                    if (lane > 0 && start <= lo - 1 && lo - 1 < end) { ta = h; oa = lo - 1 - start; }
                    start = end;
                }
            }
            sm.ha = ta; sm.hb = tb;
            if (lane > 0) {
                if (ta != tb) sm.cls = HAP_CROSS;
                else sm.cls = (oa / dc.node_size[ta] == ob / dc.node_size[tb]) ? HAP_INTRA : HAP_INTER;
            }
        }
    }
    return sm;
}

// configuration that owns candidate index c (binary search over the offsets)
__device__ __forceinline__ u64 find_pconf(const DevConst &dc, u64 c)
{
    u64 lo = 0, hi = dc.n_pconf;            // invariant: offset[lo] <= c < offset[hi] (virtual)
    while (hi - lo > 1) {
        const u64 mid = (lo + hi) >> 1;
        if (dc.pconf[mid].offset <= c) lo = mid; else hi = mid;
    }
    return lo;
}

__global__ void decode_kernel(const DevConst dc, u64 first, u64 count, hap_candidate *out, const i64 *first_dev)
{
    const u64 w = ((u64)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= count) return;
    if (first_dev) {                    // the index a preceding kernel left in device memory (negative: none)
        const i64 f = *first_dev;
        if (f < 0) return;
        first = (u64)f;
    }
    const u64 c = first + w;
    const u64 p = find_pconf(dc, c);
    const hap_pconf pc = dc.pconf[p];
    const u64 local = c - pc.offset;
    const u64 map_idx = local / (u64)dc.n_rc;
    const int rc = (int)(local - map_idx * (u64)dc.n_rc);
    const StageMap sm = decode_stage(dc, pc, map_idx, lane);
    hap_candidate *o = out + w;
    if (lane == 0) {
        o->index = c; o->pconf = (uint32_t)p; o->rc_mask = dc.rc_masks[rc]; o->map_idx = map_idx;
        o->PP = (uint8_t)pc.PP;
        for (int i = 0; i < 7; ++i) o->pad[i] = 0;
    }
    o->mask[lane] = lane < pc.PP ? (uint8_t)sm.mask : 0;
    o->link[lane] = (lane < pc.PP && lane > 0) ? (uint8_t)(sm.cls | (sm.ha << 2) | (sm.hb << 4)) : 0;
}

// Terms of one stage of a GIVEN plan (layers [a, b) at recomputation level r on the stage's device types): t_f, the
// forward time of its layers (slowest member type per layer); the stage cost c = t_f + t_b with t_b the backward
// time, the recomputed forward work and the stage constant (pre / post-processing, the transfer into the stage);
// the stage's gradient-synchronisation and optimizer times.  `stage` is 0-based.
__device__ __forceinline__ void plan_stage_terms(const DevConst &dc, u64 p, int PP, const StageMap &sm, int stage, int a, int b, int r,
                                                 const i64 *__restrict__ c2, const i64 *__restrict__ coef,
                                                 i64 &tf, i64 &cst, i64 &sy, i64 &op)
{
    const int N = dc.N, T = dc.T;
    const i64 *c2p = c2 + (size_t)p * T * N * 2;
    const i64 *cfp = coef + (size_t)p * T * HAP_NCOEF;
    i64 tb = 0;
    tf = 0;
    for (int l = a; l < b; ++l) {
        i64 F = 0, B = 0;
        for (int h = 0; h < T; ++h)
            if (sm.mask >> h & 1) {
                const i64 qx = c2p[((size_t)h * N + l) * 2], qy = c2p[((size_t)h * N + l) * 2 + 1];
                F = qx > F ? qx : F;
                B = qy > B ? qy : B;
            }
        tf += F; tb += B;
    }
    // coefficients of a stage of several types: the slowest member's
    i64 kpre = 0, kpost = 0, slat = 0, sbw[2] = {0, 0}, opt[2] = {0, 0};
    for (int h = 0; h < T; ++h)
        if (sm.mask >> h & 1) {
            const i64 *row = cfp + h * HAP_NCOEF;
            kpre = row[HAP_KPRE] > kpre ? row[HAP_KPRE] : kpre;
            kpost = row[HAP_KPOST] > kpost ? row[HAP_KPOST] : kpost;
            slat = row[HAP_SLAT] > slat ? row[HAP_SLAT] : slat;
            for (int kd = 0; kd < 2; ++kd) {
                sbw[kd] = row[HAP_SBW + kd] > sbw[kd] ? row[HAP_SBW + kd] : sbw[kd];
                opt[kd] = row[HAP_OPT + kd] > opt[kd] ? row[HAP_OPT + kd] : opt[kd];
            }
        }
    tb += ((i64)dc.tau_q[r] * tf) >> 10;              // forward work repeated in the backward pass
    if (stage == 0) tb += kpre;
    if (stage == PP - 1) tb += kpost;
    if (stage > 0) tb += cfp[sm.hb * HAP_NCOEF + (sm.cls == HAP_CROSS ? HAP_KP2P_CROSS + sm.ha : HAP_KP2P_INTRA + sm.cls)];
    cst = tf + tb;
    const i64 n_moe = (i64)(moe_before(dc, b) - moe_before(dc, a)), n_dense = (i64)(b - a) - n_moe;
    sy = slat + n_dense * sbw[0] + n_moe * sbw[1];
    op = n_dense * opt[0] + n_moe * opt[1];
}

// ------------------------------------------------------------------------------------------
// Appendix B: iteration latency of GIVEN plans with the steady-state term written through the bottleneck
// stage's index, T_middle = sum_{i <= s_max} t_f,i + max(0, M - s_max - 1) max_i (t_f,i + t_b,i), T_edge = the
// summed stage cost (Eq. 4).  t_f,i is the forward time of the stage's layers (slowest member type per layer);
// recomputation, backward time and the stage constant make up t_b,i.  One warp per candidate, lane s = stage s+1;
// partition / recompute: [count][HAP_MAX_PP] layers and levels per stage as written by the DP kernels.
// t_iter: [count]; detail: [count][3] T_edge, T_middle, s_max (nullable).
// ------------------------------------------------------------------------------------------
__global__ void appendix_b_kernel(const DevConst dc, u64 first, u64 count, const i64 *__restrict__ c2,
                                  const i64 *__restrict__ coef, const uint8_t *__restrict__ partition,
                                  const uint8_t *__restrict__ recompute, i64 *t_iter, i64 *detail)
{
    const u64 w = ((u64)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (w >= count) return;
    const u64 c = first + w;
    const u64 p = find_pconf(dc, c);
    const hap_pconf pc = dc.pconf[p];
    const int PP = pc.PP, N = dc.N;
    const u64 map_idx = (c - pc.offset) / (u64)dc.n_rc;
    const StageMap sm = decode_stage(dc, pc, map_idx, lane);
    const bool on = lane < PP;
    const int n_me = on ? partition[w * HAP_MAX_PP + lane] : 0;
    const int r_me = on ? recompute[w * HAP_MAX_PP + lane] : 0;
    int b_me = n_me;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, b_me, o); if (lane >= o) b_me += t; }
    const int total = __shfl_sync(0xffffffffu, b_me, PP - 1);
    const bool ok = total == N && !__any_sync(0xffffffffu, on && n_me == 0) && !__any_sync(0xffffffffu, on && r_me >= dc.R);
    if (!ok) {
        if (lane == 0) {
            t_iter[w] = kInf;
            if (detail) { detail[w * 3] = kInf; detail[w * 3 + 1] = kInf; detail[w * 3 + 2] = 0; }
        }
        return;
    }
    i64 tf = 0, cst = 0, sy = 0, op = 0;
    if (on) plan_stage_terms(dc, p, PP, sm, lane, b_me - n_me, b_me, r_me, c2, coef, tf, cst, sy, op);
    const i64 edge = warp_sum_i64(cst), cmax = warp_max_i64(cst);
    const i64 t_sync = warp_max_i64(sy), t_opt = warp_max_i64(op);
    const unsigned at_max = __ballot_sync(0xffffffffu, on && cst == cmax);
    const int s_lane = __ffs(at_max) - 1;                      // the first bottleneck stage
    i64 fpre = tf;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const i64 t = __shfl_up_sync(0xffffffffu, fpre, o); if (lane >= o) fpre += t; }
    const i64 f_upto = shfl_i64(fpre, s_lane);
    i64 steady = (i64)pc.M - (s_lane + 1) - 1;
    if (steady < 0) steady = 0;
    if (lane == 0) {
        const i64 middle = f_upto + steady * cmax;
        t_iter[w] = edge + middle + t_sync + t_opt;
        if (detail) { detail[w * 3] = edge; detail[w * 3 + 1] = middle; detail[w * 3 + 2] = s_lane + 1; }
    }
}

// ------------------------------------------------------------------------------------------
// Event simulation of the 1F1B schedule for GIVEN plans (the schedule whose iteration latency Eq. 4 and Appendix B
// put in closed form).  Stage i of PP (1-based) runs, in this order, min(PP - i, M) warm-up forward passes, then
// forward / backward pairs while forwards remain, then the backward passes that are left; F(i, m) starts when the
// stage is free and F(i-1, m) has ended, B(i, m) when the stage is free and B(i+1, m) has ended (last stage: its
// own F(i, m)).  A forward pass of stage i takes t_f,i, a backward pass t_b,i = c_i - t_f,i (the split of
// Appendix B), so transfers are part of the passes.  One warp per candidate, lane = stage: every round each lane runs
// its next pass if that pass's input exists; end times travel between neighbouring stages through a ring of the
// last kSimRing passes per stage and direction (a stage is at most PP passes ahead of its consumer).
// t_iter: [count] simulated pipeline time + T_sync + T_opt; detail: [count][2] simulated pipeline time and Eq. 4's
// pipeline term sum_i c_i + (M-1) max_i c_i of the same plan (nullable).
// ------------------------------------------------------------------------------------------
constexpr int kSimRing = 64;

__global__ void __launch_bounds__(32)
simulate_1f1b_kernel(const DevConst dc, u64 first, u64 count, const i64 *__restrict__ c2, const i64 *__restrict__ coef,
                     const uint8_t *__restrict__ partition, const uint8_t *__restrict__ recompute, i64 *t_iter, i64 *detail)
{
    __shared__ i64 ringF[HAP_MAX_PP][kSimRing], ringB[HAP_MAX_PP][kSimRing];
    const u64 w = blockIdx.x;
    const int lane = threadIdx.x;
    if (w >= count) return;
    const u64 c = first + w;
    const u64 p = find_pconf(dc, c);
    const hap_pconf pc = dc.pconf[p];
    const int PP = pc.PP, N = dc.N, M = pc.M;
    const u64 map_idx = (c - pc.offset) / (u64)dc.n_rc;
    const StageMap sm = decode_stage(dc, pc, map_idx, lane);
    const bool on = lane < PP;
    const int n_me = on ? partition[w * HAP_MAX_PP + lane] : 0;
    const int r_me = on ? recompute[w * HAP_MAX_PP + lane] : 0;
    int b_me = n_me;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, b_me, o); if (lane >= o) b_me += t; }
    const int total = __shfl_sync(0xffffffffu, b_me, PP - 1);
    const bool ok = total == N && M >= 1 && !__any_sync(0xffffffffu, on && n_me == 0) && !__any_sync(0xffffffffu, on && r_me >= dc.R);
    if (!ok) {
        if (lane == 0) {
            t_iter[w] = kInf;
            if (detail) { detail[w * 2] = kInf; detail[w * 2 + 1] = kInf; }
        }
        return;
    }
    i64 tf = 0, cst = 0, sy = 0, op = 0;
    if (on) plan_stage_terms(dc, p, PP, sm, lane, b_me - n_me, b_me, r_me, c2, coef, tf, cst, sy, op);
    const i64 tb = cst - tf;
    const i64 csum = warp_sum_i64(cst), cmax = warp_max_i64(cst);
    const i64 t_sync = warp_max_i64(sy), t_opt = warp_max_i64(op);

    const int warm = PP - 1 - lane < M ? PP - 1 - lane : M;
    int nf = 0, nb = 0;                     // forward / backward passes this stage has run
    i64 t_free = 0;
    // every round at least one stage runs a pass (the schedule has no cycle); the longest chain of passes is
    // 2 (M + PP), which bounds the rounds
    const int max_rounds = 4 * (M + PP) + 16;
    bool stuck = true;
    for (int round = 0; round < max_rounds; ++round) {
        const int nf_prev = __shfl_up_sync(0xffffffffu, nf, 1), nb_next = __shfl_down_sync(0xffffffffu, nb, 1);
        const bool active = on && nb < M;
        if (!__any_sync(0xffffffffu, active)) { stuck = false; break; }
        {   // a stage is never a whole ring of passes ahead of the neighbour that consumes them
            const int nf_next = __shfl_down_sync(0xffffffffu, nf, 1), nb_prev = __shfl_up_sync(0xffffffffu, nb, 1);
            (void)HAP_CHECK_OK(9, !(on && lane + 1 < PP) || nf - nf_next < kSimRing);
            (void)HAP_CHECK_OK(9, !(on && lane > 0) || nb - nb_prev < kSimRing);
            (void)nf_next; (void)nb_prev;
        }
        if (active) {
            const bool fwd = nf < M && (nf < warm || nf - nb == warm);       // the stage's next pass in its fixed order
            bool ready;
            i64 dep = 0;
            if (fwd) {
                ready = lane == 0 || nf_prev > nf;
                if (ready && lane > 0) dep = ringF[lane - 1][nf & (kSimRing - 1)];
            } else if (lane == PP - 1) {
                ready = true;                                                 // its own forward pass of the micro-batch came just before
                dep = ringF[lane][nb & (kSimRing - 1)];
            } else {
                ready = nb_next > nb;
                if (ready) dep = ringB[lane + 1][nb & (kSimRing - 1)];
            }
            if (ready) {
                const i64 start = t_free > dep ? t_free : dep;
                if (fwd) { t_free = start + tf; ringF[lane][nf & (kSimRing - 1)] = t_free; ++nf; }
                else { t_free = start + tb; ringB[lane][nb & (kSimRing - 1)] = t_free; ++nb; }
            }
        }
        __syncwarp();
    }
    const i64 end = warp_max_i64(on ? t_free : 0);
    if (lane == 0) {
        const i64 sim = stuck ? kInf : end;
        t_iter[w] = stuck ? kInf : end + t_sync + t_opt;
        if (detail) { detail[w * 2] = sim; detail[w * 2 + 1] = csum + (i64)(M - 1) * cmax; }
    }
}

// ------------------------------------------------------------------------------------------
// mapping table: decoded (mask, link) byte pairs per stage for every mapping of one PP class,
// built in every pass (and once at enumeration, for the host-side tree) so that the DP kernels do not
// unrank per candidate
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ void maptab_one(const DevConst &dc, u64 p_rep, u64 nmap, uint8_t *tab, u64 w, int lane)
{
    if (w >= nmap) return;
    const hap_pconf pc = dc.pconf[p_rep];
    const StageMap sm = decode_stage(dc, pc, w, lane);
    if (lane < pc.PP) {
        uint8_t *o = tab + (w * (u64)pc.PP + lane) * 2;
        o[0] = (uint8_t)sm.mask;
        o[1] = (uint8_t)(lane > 0 ? (sm.cls | (sm.ha << 2) | (sm.hb << 4)) : 0);
    }
}

__global__ void maptab_kernel(const DevConst dc, u64 p_rep, u64 nmap, uint8_t *tab)
{
    maptab_one(dc, p_rep, nmap, tab, ((u64)blockIdx.x * blockDim.x + threadIdx.x) >> 5, threadIdx.x & 31);
}

// The same for several PP classes in one launch (a pass decodes all classes that walk a prefix tree this way):
// class q owns blocks [blk_lo[q], blk_lo[q+1]) of 128 threads, four mappings per block.
struct DecodeJobs {
    int n;
    u32 blk_lo[HAP_MAX_PP + 2];
    u32 p_rep[HAP_MAX_PP + 1];
    u32 nmap[HAP_MAX_PP + 1];
    u64 tab_off[HAP_MAX_PP + 1];            // byte offset of the class's table
};

__global__ void __launch_bounds__(128) maptab_all_kernel(const DevConst dc, const DecodeJobs jobs, uint8_t *tab_base)
{
    int q = 0;
    while (q + 1 < jobs.n && blockIdx.x >= jobs.blk_lo[q + 1]) ++q;
    const u64 w = ((u64)(blockIdx.x - jobs.blk_lo[q]) * blockDim.x + threadIdx.x) >> 5;
    maptab_one(dc, jobs.p_rep[q], jobs.nmap[q], tab_base + jobs.tab_off[q], w, threadIdx.x & 31);
}

// ------------------------------------------------------------------------------------------
// pipeline DP
// ------------------------------------------------------------------------------------------
// Shared memory of one block (all candidates of a block belong to one configuration):
//   sR   [mask rows][RW][N+1]  i64 prefix sums of stage time per type mask.  LINEAR (every tau_q a
//                              multiple of 1024): one row per recomputation level r holding
//                              fwd+bwd + (tau_r/1024)*fwd, so a span costs one subtraction; otherwise
//                              two rows (fwd+bwd, fwd) and the general formula.  Homogeneous (multiset)
//                              configurations keep one mask row per device type, block mode one per mask.
//   sW, sA [N+1]               i64 prefix sums of weight bytes / activation bytes per micro-batch
//   thr  [PP][T][R][N+1]       u8: first split k for which stage i on a device of capacity type t
//                              fits layers (k, j] at recomputation level r (j = none)
//   sK   [N+1]                 u8: number of MoE layers among the first l layers
//   per warp: rows [PP][N+1] i64 (one DP row per stage, kept so that the next mapping can reuse the rows
//             of the stage prefix it shares), ch [PP][N+1] u8 split choices
__host__ __device__ inline size_t dp_smem_bytes(int N, int PP, int T, int R, int warps, bool multiset, bool linear,
                                                bool refine = false)
{
    const size_t n1 = (size_t)N + 1;
    const size_t mrows = multiset ? (size_t)T : (size_t)((1 << T) - 1);
    size_t b = mrows * (linear ? (size_t)R : 2) * n1 * 8 + n1 * 16;
    b += ((size_t)PP * T * R * n1 + 15) / 16 * 16;
    b += (n1 + 15) / 16 * 16;
    const size_t nrows = multiset ? (size_t)PP : (size_t)(PP < 2 ? PP : 2);   // rows are reused only across multiset mappings
    b += (size_t)warps * ((nrows * n1 * 8) + (((size_t)PP * n1 + 15) / 16 * 16));
    if (refine) b += (size_t)warps * 2 * n1 * 8;             // two rotating rows of the second (additive) pass
    return b + 32;
}

template <typename VT>
struct StagePar {
    int mrow, capt;             // row of the stage's type mask in sR; index of the type whose capacity binds
    VT K;                       // stage constant: pre/post work + p2p transfer into the stage
    int nmin, nmax;             // load-balance window on the layer count
    int bl, bh;                 // band of end layers j that can be reached at this stage
};

__device__ __forceinline__ bool span_fits(const i64 *sW, const i64 *sA, const uint8_t *sK, i64 extra, i64 mx,
                                          i64 mstore, i64 cap, i64 xi, int a, int b)
{
    const bool has_moe = sK[b] != sK[a];
    const i64 Wb = (sW[b] - sW[a]) + extra + (has_moe ? mx : 0);
    const i64 A = mstore * (sA[b] - sA[a]);
    return Wb + ((xi * A) >> 10) <= cap;               // A >= 0: the shift is the floor division by 1024
}

// value type of the times: int64 (rounded ns, exact arithmetic) or double (fp64 mode)
template <typename VT> struct ValInf;
template <> struct ValInf<i64> { static __device__ __forceinline__ i64 get() { return kInf; } };
template <> struct ValInf<double> { static __device__ __forceinline__ double get() { return __longlong_as_double(0x7ff0000000000000ll); } };

template <typename VT> __device__ __forceinline__ VT shfl_v(VT v, int src) { return __shfl_sync(0xffffffffu, v, src); }

// forward-recomputation time: floor(tau * F / 1024) on integers (F >= 0), (tau / 1024.0) * F in fp64 mode
__device__ __forceinline__ i64 tau_term(i64 tau, i64 F) { return (tau * F) >> 10; }
__device__ __forceinline__ double tau_term(i64 tau, double F) { return ((double)tau / 1024.0) * F; }

// per type mask: what a stage made of these device types costs beyond its layers (slowest member),
// which member's memory binds, and the slowest member's compute rate for the load-balance window
template <typename VT>
struct MaskInfo {
    VT kpre, kpost, slat, sbw[2], opt[2];
    VT kxd;             // what an MoE layer of a stage with these types adds to the cross-type time of Pruning 3 (0: one type, or option off)
    i64 Pmin;
    int capt, pad;
};

// Block prologue shared by the DP kernels: everything that depends on the configuration only.
// All threads of the block call it; it ends with a barrier.
// Part 1: stage-time prefix rows per type mask, byte prefixes, per-mask stage info, p2p coefficients.
template <typename VT, bool LINEAR>
__device__ __forceinline__ void dp_prologue_rows(
    const DevConst &dc, unsigned p_index, const VT *c2, const i64 *coef, const VT *coefv,
    bool multiset, int mrows, int RW, unsigned masks_used, int nwarps,
    VT *sR, i64 *sW, i64 *sA, uint8_t *sK, MaskInfo<VT> *minfo, VT (*sP2P)[6], VT *szero)
{
    const int N = dc.N, T = dc.T, R = dc.R, n1 = N + 1;
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int nmask = (1 << T) - 1;
    // ---- block prologue 1: rows of this configuration -----------------------------------
    const VT *c2p = c2 + (size_t)p_index * T * N * 2;
    const i64 *cfp = coef + (size_t)p_index * T * HAP_NCOEF;
    const VT *cvp = coefv + (size_t)p_index * T * HAP_NCOEF;
    for (int mr = wib; mr < mrows; mr += nwarps) {
        // time rows of one type mask: per layer the slowest member type, then prefix sums
        const int mk = multiset ? (1 << mr) : mr + 1;
        if (!((masks_used >> mk) & 1u)) continue;                   // no mapping of this class has such a stage
        VT runC = 0, runF = 0;
        for (int base = 0; base < N; base += 32) {
            const int l = base + lane;
            VT vC = 0, vF = 0;
            if (l < N) {
                VT F = 0, B = 0;
                for (int h = 0; h < T; ++h)
                    if (mk >> h & 1) {
                        const VT qx = c2p[((size_t)h * N + l) * 2], qy = c2p[((size_t)h * N + l) * 2 + 1];
                        F = qx > F ? qx : F;
                        B = qy > B ? qy : B;
                    }
                vC = F + B; vF = F;
            }
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {      // inclusive warp scan
                const VT tC = __shfl_up_sync(0xffffffffu, vC, o), tF = __shfl_up_sync(0xffffffffu, vF, o);
                if (lane >= o) { vC += tC; vF += tF; }
            }
            vC += runC; vF += runF;
            if (l < N) {
                if (LINEAR) {
                    for (int r = 0; r < R; ++r) sR[((size_t)mr * RW + r) * n1 + l + 1] = vC + (VT)(dc.tau_q[r] >> 10) * vF;
                } else {
                    sR[((size_t)mr * RW) * n1 + l + 1] = vC; sR[((size_t)mr * RW + 1) * n1 + l + 1] = vF;
                }
            }
            runC = shfl_v(vC, 31); runF = shfl_v(vF, 31);
        }
        if (lane == 0) for (int r = 0; r < RW; ++r) sR[((size_t)mr * RW + r) * n1] = 0;
    }
    if (wib == mrows % nwarps) {
        // byte rows (integers in both modes): weights and activations per layer kind, prefix sums
        i64 runW = 0, runA = 0;
        for (int base = 0; base < N; base += 32) {
            const int l = base + lane;
            i64 vW = 0, vA = 0;
            if (l < N) { const int kd = layer_kind(dc, l); vW = cfp[HAP_MW + kd]; vA = cfp[HAP_MA + kd]; }
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const i64 tW = __shfl_up_sync(0xffffffffu, vW, o), tA = __shfl_up_sync(0xffffffffu, vA, o);
                if (lane >= o) { vW += tW; vA += tA; }
            }
            vW += runW; vA += runA;
            if (l < N) { sW[l + 1] = vW; sA[l + 1] = vA; }
            runW = shfl_i64(vW, 31); runA = shfl_i64(vA, 31);
        }
        if (lane == 0) { sW[0] = 0; sA[0] = 0; }
    }
    for (int l = threadIdx.x; l <= N; l += nwarps * 32) sK[l] = (uint8_t)moe_before(dc, l);
    if (threadIdx.x < nmask) {
        const int mk = threadIdx.x + 1;
        MaskInfo<VT> mi;
        mi.kpre = mi.kpost = mi.slat = mi.sbw[0] = mi.sbw[1] = mi.opt[0] = mi.opt[1] = 0; mi.kxd = 0; mi.Pmin = 0; mi.capt = 0; mi.pad = 0;
        i64 cap = 0;
        bool seen = false;
        const bool het_stage = dc.het_dispatch && (mk & (mk - 1)) != 0;      // more than one device type
        for (int h = 0; h < T; ++h)
            if (mk >> h & 1) {
                const VT *row = cvp + h * HAP_NCOEF;
                if (het_stage && row[HAP_KXD] > mi.kxd) mi.kxd = row[HAP_KXD];
                if (!seen || dc.cap_eff[h] < cap) { cap = dc.cap_eff[h]; mi.capt = h; }
                if (!seen || dc.P[h] < mi.Pmin) mi.Pmin = dc.P[h];
                if (!seen || row[HAP_KPRE] > mi.kpre) mi.kpre = row[HAP_KPRE];
                if (!seen || row[HAP_KPOST] > mi.kpost) mi.kpost = row[HAP_KPOST];
                if (!seen || row[HAP_SLAT] > mi.slat) mi.slat = row[HAP_SLAT];
                if (!seen || row[HAP_SBW] > mi.sbw[0]) mi.sbw[0] = row[HAP_SBW];
                if (!seen || row[HAP_SBW + 1] > mi.sbw[1]) mi.sbw[1] = row[HAP_SBW + 1];
                if (!seen || row[HAP_OPT] > mi.opt[0]) mi.opt[0] = row[HAP_OPT];
                if (!seen || row[HAP_OPT + 1] > mi.opt[1]) mi.opt[1] = row[HAP_OPT + 1];
                seen = true;
            }
        minfo[threadIdx.x] = mi;
    }
    if (threadIdx.x >= 32 && threadIdx.x < 32 + T * 6) {
        const int q = threadIdx.x - 32, h = q / 6, e = q % 6;
        sP2P[h][e] = cvp[h * HAP_NCOEF + HAP_KP2P_INTRA + e];      // intra, inter, cross[0..3] are consecutive columns
    }
    if (threadIdx.x == 0) szero[0] = 0;
    __syncthreads();
}

// Part 2: memory-threshold tables and the per-type load-balance window.
template <typename VT>
__device__ __forceinline__ void dp_prologue_thr(
    const DevConst &dc, const hap_pconf &pc, unsigned p_index, const i64 *coef, bool multiset, int nwarps,
    const i64 *sW, const i64 *sA, uint8_t *thr, const uint8_t *sK, int (*winT)[2])
{
    const int N = dc.N, T = dc.T, R = dc.R, n1 = N + 1, PP = pc.PP;
    const i64 *cfp = coef + (size_t)p_index * T * HAP_NCOEF;
    // ---- block prologue 2: memory thresholds ----------------------------------------------
    // Feasibility of a span (k, j] is monotone: a shorter span needs no more memory, and the first
    // feasible k does not decrease with j.  One thread sweeps j for one (stage, capacity type, level).
    const i64 mx = cfp[HAP_MX], mpre = cfp[HAP_MPRE], mpost = cfp[HAP_MPOST];
    const int combos = PP * T * R, nthreads = nwarps * 32;
    if (combos * 7 < nthreads * 2) {
        // few (stage, type, level) rows for this many threads: one thread per table entry, binary search over k
        for (int e = threadIdx.x; e < combos * n1; e += nthreads) {
            const int q = e / n1, j = e - q * n1;
            const int r = q % R, t = (q / R) % T, i = q / (R * T) + 1;
            const i64 extra = (i == 1 ? mpre : 0) + (i == PP ? mpost : 0);
            const int inflight = PP - i + 1;
            const i64 mstore = pc.M < inflight ? pc.M : inflight;
            const i64 cap = dc.cap_eff[t], xi = dc.xi_q[r];
            int lo = 0, hi = j;                       // first k in [0, j] whose span (k, j] fits; j if none
            while (lo < hi) {
                const int mid = (lo + hi) >> 1;
                if (span_fits(sW, sA, sK, extra, mx, mstore, cap, xi, mid, j)) hi = mid; else lo = mid + 1;
            }
            thr[(size_t)q * n1 + j] = (uint8_t)lo;
        }
    } else {
        for (int q = threadIdx.x; q < combos; q += nthreads) {
            const int r = q % R, t = (q / R) % T, i = q / (R * T) + 1;
            const i64 extra = (i == 1 ? mpre : 0) + (i == PP ? mpost : 0);
            const int inflight = PP - i + 1;
            const i64 mstore = pc.M < inflight ? pc.M : inflight;
            const i64 cap = dc.cap_eff[t], xi = dc.xi_q[r];
            uint8_t *row = thr + (size_t)q * n1;
            int k = 0;
            row[0] = 0;
            for (int j = 1; j <= N; ++j) {
                while (k < j && !span_fits(sW, sA, sK, extra, mx, mstore, cap, xi, k, j)) ++k;
                row[j] = (uint8_t)k;
            }
        }
    }
    // load-balance window per device type when every mapping uses the same multiset of stage types
    if (threadIdx.x < T) {
        int lo = 1, hi = N - PP + 1;
        if (dc.delta_q >= 0 && multiset) {
            i64 Ps = 0;
            for (int h = 0; h < T; ++h) Ps += (dc.m[h] / pc.G) * dc.P[h];
            const i64 den = 1024 * Ps, Ph = dc.P[threadIdx.x];
            i64 a = ((i64)(1024 - dc.delta_q) * Ph * N) / den;
            i64 b = ((i64)(1024 + dc.delta_q) * Ph * N + den - 1) / den;
            lo = a < 1 ? 1 : (int)a;
            hi = b > N - PP + 1 ? N - PP + 1 : (int)b;
        }
        if (dc.uniform) { lo = N / PP; hi = (N + PP - 1) / PP; }      // ablation: uniform layer split only
        winT[threadIdx.x][0] = lo; winT[threadIdx.x][1] = hi;
    }
    __syncthreads();
}

template <typename VT, bool LINEAR>
__device__ __forceinline__ void dp_block_prologue(
    const DevConst &dc, const hap_pconf &pc, unsigned p_index, const VT *c2, const i64 *coef, const VT *coefv,
    bool multiset, int mrows, int RW, unsigned masks_used, int nwarps,
    VT *sR, i64 *sW, i64 *sA, uint8_t *thr, uint8_t *sK, MaskInfo<VT> *minfo, VT (*sP2P)[6], VT *szero, int (*winT)[2])
{
    dp_prologue_rows<VT, LINEAR>(dc, p_index, c2, coef, coefv, multiset, mrows, RW, masks_used, nwarps,
                                 sR, sW, sA, sK, minfo, sP2P, szero);
    dp_prologue_thr<VT>(dc, pc, p_index, coef, multiset, nwarps, sW, sA, thr, sK, winT);
}

// two blocks of up to 12 warps per SM: the register cap (85) keeps the occupancy independent of ptxas' heuristics
template <bool SEARCH, bool LINEAR, bool COUNT = false, typename VT = i64, bool REFINE = false>
__global__ void __launch_bounds__(kDpWarps * 32, 2)
pipeline_dp_kernel(const DevConst dc, const WorkItem *items, const VT *c2, const i64 *coef, const VT *coefv,
                   const uint8_t *maptab, DpOut out, int nwarps, unsigned masks_used)
{
    // c2: layer times; coef: integer coefficients (memory bytes); coefv: time coefficients in the value type
    // (the same array as coef in integer mode)
    const VT vInf = ValInf<VT>::get();
    if (out.first_dev) {
        // the range starts at an index a preceding kernel left in device memory (the winner of a search)
        const i64 f = *out.first_dev;
        out.first = f < 0 ? (~0ull >> 1) : (u64)f;
    }
    extern __shared__ __align__(16) unsigned char smem_raw[];
    const int N = dc.N, T = dc.T, R = dc.R, n1 = N + 1;
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const WorkItem it = items[blockIdx.x];
    const hap_pconf pc = dc.pconf[it.p];
    const int PP = pc.PP, n_rc = dc.n_rc;
    {   // blocks whose candidates all lie outside the requested range have nothing to do
        const u64 c0 = pc.offset + it.lo * (u64)n_rc, c1 = c0 + (u64)it.count * n_rc;
        if (c1 <= out.first || c0 >= out.first + out.count) {
            if (SEARCH && threadIdx.x == 0) { out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull; }
            return;
        }
    }
    if (SEARCH && out.prune) {
        // T_iter >= sum_i c_i + (M-1) max_i c_i >= S + (M-1) ceil(S / PP) with S the configuration's lower bound on
        // the summed stage time.  Skipping needs bound > incumbent (strict): the result cannot change.
        // The incumbent moves while the block runs, so ONE thread reads it and the whole block follows that
        // reading: a block must leave as a whole.
        __shared__ int s_skip;
        if (threadIdx.x == 0) {
            const i64 S = out.lb_sum[it.p];
            const i64 lb = S + (i64)(pc.M - 1) * ((S + PP - 1) / PP);
            const u64 inc = *reinterpret_cast<volatile const u64 *>(out.incumbent);
            s_skip = (u64)lb > inc;
            if (s_skip) {
                out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull;
                // candidates of this block inside the requested range
                const u64 c0 = pc.offset + it.lo * (u64)n_rc, c1 = c0 + (u64)it.count * n_rc;
                const u64 a = c0 > out.first ? c0 : out.first, b = c1 < out.first + out.count ? c1 : out.first + out.count;
                atomicAdd(out.counters + 2, b - a);
            }
        }
        __syncthreads();
        if (s_skip) return;
    }
    if (SEARCH && out.cand_lb) {
        // bounds of the block's candidates against the incumbent: when none can win, the block leaves before its prologue
        const u64 c0 = pc.offset + it.lo * (u64)n_rc, c1 = c0 + (u64)it.count * n_rc;
        const u64 a = c0 > out.first ? c0 : out.first, b = c1 < out.first + out.count ? c1 : out.first + out.count;
        const u64 inc = *reinterpret_cast<volatile const u64 *>(out.incumbent);
        int alive = 0;
        u64 n_inf = 0, n_cut = 0;
        for (u64 c = a + threadIdx.x; c < b; c += blockDim.x) {
            const i64 lb = out.cand_lb[c];
            if (lb >= kInf) n_inf++;
            else if ((u64)lb > inc) n_cut++;
            else alive = 1;
        }
        if (!__syncthreads_or(alive)) {
            n_inf = (u64)warp_sum_i64((i64)n_inf); n_cut = (u64)warp_sum_i64((i64)n_cut);
            if (lane == 0) {
                if (n_inf) atomicAdd(out.counters + 0, n_inf);
                if (n_cut) atomicAdd(out.counters + 2, n_cut);
            }
            if (threadIdx.x == 0) { out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull; }
            return;
        }
    }
    const bool multiset = pc.mode == HAP_MAP_MULTISET;
    const int nmask = (1 << T) - 1;
    const int mrows = multiset ? T : nmask;
    const int RW = LINEAR ? R : 2;

    VT *sR = reinterpret_cast<VT *>(smem_raw);
    i64 *sW = reinterpret_cast<i64 *>(sR + (size_t)mrows * RW * n1);
    i64 *sA = sW + n1;
    uint8_t *thr = reinterpret_cast<uint8_t *>(sA + n1);
    const size_t thr_bytes = ((size_t)PP * T * R * n1 + 15) / 16 * 16;
    uint8_t *sK = thr + thr_bytes;
    const int nrows = multiset ? PP : (PP < 2 ? PP : 2);   // block mode shares nothing between mappings: two rotating rows
    const size_t row_bytes = (size_t)nrows * n1 * 8, ch_bytes = ((size_t)PP * n1 + 15) / 16 * 16;
    unsigned char *wbase = sK + ((size_t)n1 + 15) / 16 * 16 + (size_t)wib * (row_bytes + ch_bytes);
    VT *rows = reinterpret_cast<VT *>(wbase);            // row of stage i at rows + ((i-1) % nrows)*n1
    uint8_t *chw = wbase + row_bytes;
    // second-pass rows (refinement) sit behind all warps' first-pass storage
    VT *rows2 = reinterpret_cast<VT *>(sK + ((size_t)n1 + 15) / 16 * 16 + (size_t)nwarps * (row_bytes + ch_bytes)) + (size_t)wib * 2 * n1;
    __shared__ MaskInfo<VT> minfo[kMaxMasks];
    __shared__ VT sP2P[HAP_MAX_TYPES][6];                 // per receiving type: intra, inter, cross from type 0..3
    __shared__ VT szero[1];                               // the row of "stage 0": DP[0][0] = 0
    __shared__ int winT[HAP_MAX_TYPES][2];

    dp_block_prologue<VT, LINEAR>(dc, pc, it.p, c2, coef, coefv, multiset, mrows, RW, masks_used, nwarps,
                                  sR, sW, sA, thr, sK, minfo, sP2P, szero, winT);

    VT best_cost = vInf;
    u64 best_index = ~0ull;
    u64 n_eval = 0, n_feas = 0, n_cells = 0;
    const bool want_tables = !SEARCH && (out.dp_table != nullptr || out.choice != nullptr);
    int red0 = 1;                                    // reductions over the stages span the next power of two >= PP lanes
    while (red0 < PP) red0 <<= 1;
    red0 >>= 1;

    // warp -> slice of consecutive mappings, evaluated once per recompute policy.  Consecutive mappings share a
    // prefix of stage types, and the DP rows of a shared prefix are reused.  Policies run from the most
    // permissive to the most restrictive (dc.rc_order): a mapping that admits no feasible partition under a
    // policy admits none under any policy whose allowed levels are a subset, so it is skipped there.
    __shared__ u64 s_infeas[kDpWarps][HAP_MAX_RC_MASKS];
    const u32 per_slice = (it.count + nwarps - 1) / nwarps;          // <= 64 (host chunking)
    for (int rc_pos = 0; rc_pos < n_rc; ++rc_pos) {
      const int rc_idx = dc.rc_order[rc_pos];
      const unsigned rc_mask = dc.rc_masks[rc_idx];
      const u32 m_lo = (u32)wib * per_slice;
      const u32 m_hi = m_lo + per_slice < it.count ? m_lo + per_slice : it.count;
      u64 known_infeasible = 0, infeasible_here = 0;
      if (!COUNT && !want_tables)
          for (int q = 0; q < rc_pos; ++q)
              if ((dc.rc_sup[rc_pos] >> q) & 1u) known_infeasible |= s_infeas[wib][q];
      int valid_rows = 0;                  // DP rows of stages 1..valid_rows of the previous mapping are intact
      int dead_stage = 1 << 30;            // first of those stages whose row holds no finite value (none: large)
      int prev_mask = -1, prev_link = -1;
      uchar2 next_ml = make_uchar2(0, 0);
      if (maptab && m_lo < m_hi && lane < PP)
          next_ml = *reinterpret_cast<const uchar2 *>(maptab + ((it.lo + m_lo) * (u64)PP + lane) * 2);
      for (u32 mi = m_lo; mi < m_hi; ++mi) {
        const u64 map_idx = it.lo + mi;
        const u64 c = pc.offset + map_idx * (u64)n_rc + (u64)rc_idx;

        // ---- stage types of this mapping, lane s holds stage s+1 -----------------------------
        int mask = 0, link = 0;
        if (maptab) {
            mask = next_ml.x; link = next_ml.y;
            if (mi + 1 < m_hi && lane < PP)        // fetch the next mapping while this one is evaluated
                next_ml = *reinterpret_cast<const uchar2 *>(maptab + ((map_idx + 1) * (u64)PP + lane) * 2);
        } else {
            const StageMap smap = decode_stage(dc, pc, map_idx, lane);
            mask = smap.mask; link = lane > 0 && lane < PP ? (smap.cls | (smap.ha << 2) | (smap.hb << 4)) : 0;
        }
        if (c < out.first || c >= out.first + out.count) { valid_rows = 0; dead_stage = 1 << 30; prev_mask = -1; continue; }
        if (SEARCH && out.cand_lb) {
            // the candidate's lower bound from the plain pass (one address for the whole warp, so one reading)
            const i64 lb = out.cand_lb[c];
            const u64 inc = *reinterpret_cast<volatile const u64 *>(out.incumbent);
            if (lb >= kInf || (u64)lb > inc) {
                valid_rows = 0; dead_stage = 1 << 30; prev_mask = -1;
                if (lb >= kInf) n_eval++;
                else if (lane == 0) atomicAdd(out.counters + 2, 1ull);
                continue;
            }
        }
        if ((known_infeasible >> (mi - m_lo)) & 1ull) {
            // infeasible under a more permissive policy: infeasible here, nothing to compute
            infeasible_here |= 1ull << (mi - m_lo);
            valid_rows = 0; dead_stage = 1 << 30; prev_mask = -1;
            if (SEARCH) n_eval++;
            else {
                const u64 o = c - out.first;
                if (lane == 0) {
                    if (out.cost) reinterpret_cast<VT *>(out.cost)[o] = vInf;
                    if (out.bottleneck) reinterpret_cast<VT *>(out.bottleneck)[o] = vInf;
                    if (out.detail) { VT *d = reinterpret_cast<VT *>(out.detail); d[o * 3] = vInf; d[o * 3 + 1] = 0; d[o * 3 + 2] = 0; }
                }
                if (out.partition) out.partition[o * HAP_MAX_PP + lane] = 0;
                if (out.recompute) out.recompute[o * HAP_MAX_PP + lane] = 0;
            }
            continue;
        }
        const unsigned differ = __ballot_sync(0xffffffffu, lane < PP && (mask != prev_mask || link != prev_link));
        int s0 = differ ? __ffs(differ) - 1 : PP;      // stages 1..s0 are shared with the previous mapping
        prev_mask = mask; prev_link = link;
        if (!multiset) s0 = 0;               // block mode: window and bands depend on the whole mapping
        if (s0 > valid_rows) s0 = valid_rows;
        if (want_tables) s0 = 0;
        if (dead_stage > s0) dead_stage = 1 << 30;       // the dead row, if any, is not part of the shared prefix
        if (!COUNT && dead_stage <= s0) {
            // a shared stage prefix that already admits no feasible partition settles this mapping too
            valid_rows = s0;
            infeasible_here |= 1ull << (mi - m_lo);
            if (SEARCH) n_eval++;
            else {
                const u64 o = c - out.first;
                if (lane == 0) {
                    if (out.cost) reinterpret_cast<VT *>(out.cost)[o] = vInf;
                    if (out.bottleneck) reinterpret_cast<VT *>(out.bottleneck)[o] = vInf;
                    if (out.detail) { VT *d = reinterpret_cast<VT *>(out.detail); d[o * 3] = vInf; d[o * 3 + 1] = 0; d[o * 3 + 2] = 0; }
                }
                if (out.partition) out.partition[o * HAP_MAX_PP + lane] = 0;
                if (out.recompute) out.recompute[o * HAP_MAX_PP + lane] = 0;
            }
            continue;
        }

        StagePar<VT> sp;
        sp.mrow = 0; sp.capt = 0; sp.K = 0; sp.nmin = 1; sp.nmax = N - PP + 1; sp.bl = 0; sp.bh = 0;
        i64 Pmin = 0;
        if (lane < PP) {
            const MaskInfo<VT> &mi_ = minfo[mask - 1];
            sp.mrow = multiset ? __ffs(mask) - 1 : mask - 1;
            sp.capt = mi_.capt; Pmin = mi_.Pmin;
            if (lane == 0) sp.K += mi_.kpre;
            if (lane == PP - 1) sp.K += mi_.kpost;
            if (lane > 0) {
                const int cls = link & 3, ha = (link >> 2) & 3, hb = (link >> 4) & 3;
                sp.K += sP2P[hb][cls == HAP_CROSS ? 2 + ha : cls];
            }
        }
        if (dc.uniform) {
            if (lane < PP) { sp.nmin = N / PP; sp.nmax = (N + PP - 1) / PP; }
        } else if (dc.delta_q >= 0) {
            if (multiset) {
                if (lane < PP) { sp.nmin = winT[sp.mrow][0]; sp.nmax = winT[sp.mrow][1]; }   // homogeneous stage: its one type
            } else {
                const i64 Ps = warp_sum_i64(lane < PP ? Pmin : 0);
                if (lane < PP) {
                    const i64 den = 1024 * Ps;
                    i64 lo = ((i64)(1024 - dc.delta_q) * Pmin * N) / den;
                    i64 hi = ((i64)(1024 + dc.delta_q) * Pmin * N + den - 1) / den;
                    if (lo < 1) lo = 1;
                    if (hi > N - PP + 1) hi = N - PP + 1;
                    sp.nmin = (int)lo; sp.nmax = (int)hi;
                }
            }
        }
        // ---- bands: end layers j that stage i can reach (prefix sums of the window bounds), and from
        //      which the remaining stages can still reach N (suffix sums; not applied when the caller
        //      wants the full tables, where such cells hold finite values)
        {
            int smin = lane < PP ? sp.nmin : 0, smax = lane < PP ? sp.nmax : 0;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int a = __shfl_up_sync(0xffffffffu, smin, o), b = __shfl_up_sync(0xffffffffu, smax, o);
                if (lane >= o) { smin += a; smax += b; }
            }
            const int tmin = __shfl_sync(0xffffffffu, smin, PP - 1), tmax = __shfl_sync(0xffffffffu, smax, PP - 1);
            const int i = lane + 1;
            int bl = smin > i ? smin : i, bh = smax < N - PP + i ? smax : N - PP + i;
            if (!want_tables) {
                const int rl = N - (tmax - smax), rh = N - (tmin - smin);   // remaining stages take [tmin-smin, tmax-smax]
                bl = bl > rl ? bl : rl; bh = bh < rh ? bh : rh;
            }
            sp.bl = bl; sp.bh = bh;
        }
        const bool dead = __any_sync(0xffffffffu, lane < PP && sp.bl > sp.bh);
        if (COUNT) {
            dead_stage = 1 << 30;
            // cells (i, j, k) of this candidate's recurrence whose stage cost is finite: k inside the load-balance
            // window of stage i and the span (k, j] within the memory limit at some allowed level
            for (int i = 1; i <= PP; ++i) {
                const int src = i - 1;
                const int capt = __shfl_sync(0xffffffffu, sp.capt, src);
                const int nmin = __shfl_sync(0xffffffffu, sp.nmin, src), nmax = __shfl_sync(0xffffffffu, sp.nmax, src);
                const uint8_t *th = thr + ((size_t)(i - 1) * T + capt) * R * n1;
                for (int j = i + lane; j <= N - PP + i; j += 32) {
                    int klo = j - nmax; if (klo < i - 1) klo = i - 1;
                    const int khi = j - nmin;
                    int kf = 255;
                    for (int r = 0; r < R; ++r)
                        if ((rc_mask >> r) & 1u) { const int t = th[(size_t)r * n1 + j]; kf = t < kf ? t : kf; }
                    if (kf > klo) klo = kf;
                    if (klo <= khi) n_cells += (u64)(khi - klo + 1);
                }
            }
            valid_rows = 0;
            continue;
        }

        // ---- recurrence -------------------------------------------------------------------
        VT *tab_out = nullptr; uint8_t *ch_out = nullptr;
        if (want_tables) {
            if (out.dp_table) tab_out = reinterpret_cast<VT *>(out.dp_table) + (size_t)(c - out.first) * (HAP_MAX_PP + 1) * n1;
            if (out.choice) ch_out = out.choice + (size_t)(c - out.first) * (HAP_MAX_PP + 1) * n1;
            for (int j = lane; j <= N; j += 32) {
                if (tab_out) tab_out[j] = j == 0 ? (VT)0 : vInf;
                if (ch_out) ch_out[j] = 255;
            }
        }
        VT bott = vInf;
        if (!dead || want_tables) {
            int pbl = 0, pbh = 0;                          // band of the previous stage (stage 0: {0})
            int last_stage = PP;
            if (s0 > 0) { pbl = __shfl_sync(0xffffffffu, sp.bl, s0 - 1); pbh = __shfl_sync(0xffffffffu, sp.bh, s0 - 1); }
            for (int i = s0 + 1; i <= PP; ++i) {
                const int src = i - 1;
                const int mrow = __shfl_sync(0xffffffffu, sp.mrow, src), capt = __shfl_sync(0xffffffffu, sp.capt, src);
                const VT K = shfl_v(sp.K, src);
                const int nmin = __shfl_sync(0xffffffffu, sp.nmin, src), nmax = __shfl_sync(0xffffffffu, sp.nmax, src);
                const int bl = __shfl_sync(0xffffffffu, sp.bl, src), bh = __shfl_sync(0xffffffffu, sp.bh, src);
                const VT *rM = sR + (size_t)mrow * RW * n1;
                const int ri = multiset ? i - 1 : (i - 1) & 1;          // two rotating rows in block mode
                const VT *prev = i == 1 ? szero : rows + (multiset ? ri - 1 : ri ^ 1) * n1;
                VT *cur = rows + ri * n1;
                uint8_t *chrow = chw + (size_t)(i - 1) * n1;
                const uint8_t *th = thr + ((size_t)(i - 1) * T + capt) * R * n1;
                bool row_alive = false;
                for (int j = bl + lane; j <= bh; j += 32) {
                    VT best = vInf;
                    int arg = 255;
                    int klo = j - nmax; if (klo < pbl) klo = pbl;
                    int khi = j - nmin; if (khi > pbh) khi = pbh;
                    if (klo <= khi) {
                        int seg_hi = khi;                     // k range still to be assigned a level
                        for (int r = 0; r < R && seg_hi >= klo; ++r) {
                            if (!((rc_mask >> r) & 1u)) continue;
                            int lo = th[(size_t)r * n1 + j];   // first k that fits at level r
                            if (lo < klo) lo = klo;
                            if (lo > seg_hi) continue;
                            n_cells += (u64)(seg_hi - lo + 1);
                            if (LINEAR) {
                                const VT *rr = rM + (size_t)r * n1;
                                const VT Cj = rr[j] + K;
                                for (int k = seg_hi; k >= lo; --k) {
                                    const VT pv = prev[k];
                                    const VT cst = Cj - rr[k];
                                    const VT v = pv > cst ? pv : cst;
                                    if (v <= best && v < vInf) { best = v; arg = k; }   // descending k, <=: smallest k wins
                                    // layer times are non-negative: the stage cost only grows as k falls within a
                                    // level, so no further split of this level can reach the best value
                                    if (cst > best) break;
                                }
                            } else {
                                const VT *rC = rM, *rF = rM + n1;
                                const VT Cj = rC[j] + K, Fj = rF[j];
                                const i64 tau = dc.tau_q[r];
                                for (int k = seg_hi; k >= lo; --k) {
                                    const VT pv = prev[k];
                                    const VT cst = (Cj - rC[k]) + tau_term(tau, Fj - rF[k]);   // forward sums are non-negative
                                    const VT v = pv > cst ? pv : cst;
                                    if (v <= best && v < vInf) { best = v; arg = k; }
                                    if (cst > best) break;
                                }
                            }
                            seg_hi = lo - 1;
                        }
                    }
                    cur[j] = best;
                    chrow[j] = (uint8_t)arg;
                    row_alive |= best < vInf;
                }
                __syncwarp();
                if (!want_tables && !__any_sync(0xffffffffu, row_alive)) {
                    // no end layer of this stage is reachable within the memory limit: the candidate and every
                    // mapping that shares stages 1..i with it are infeasible
                    dead_stage = i;
                    last_stage = i;
                    break;
                }
                if (want_tables) {
                    for (int j = lane; j <= N; j += 32) {
                        const bool in = j >= bl && j <= bh;
                        if (tab_out) tab_out[(size_t)i * n1 + j] = in ? cur[j] : vInf;
                        if (ch_out) ch_out[(size_t)i * n1 + j] = in ? chrow[j] : (uint8_t)255;
                    }
                }
                pbl = bl; pbh = bh;
            }
            valid_rows = dead ? 0 : last_stage;
            // N lies in the last band unless the windows cannot add up to N (possible only without the
            // suffix restriction, i.e. when tables are written)
            if (!dead && dead_stage > PP && pbl <= N && N <= pbh) bott = rows[(size_t)(multiset ? PP - 1 : (PP - 1) & 1) * n1 + N];
        } else {
            valid_rows = 0;
        }
        __syncwarp();

        if (!(bott < vInf)) infeasible_here |= 1ull << (mi - m_lo);
        int ref_a = 0, ref_b = 0;                          // refinement: this lane's stage span of the chosen partition
        if (REFINE && bott < vInf) {
            // ---- refinement: an additive recurrence over the same bands with a limit on the stage cost.
            //      limit = bottleneck: the smallest stage-cost sum among the bottleneck-optimal partitions.
            //      exact mode: the limit is then swept upward over the stage costs that were skipped, which
            //      reaches the optimum of sum + (M-1) max over all partitions (see below).
            //      The first pass's rows stay intact for the next mapping; the split choices are overwritten.
            const VT M1 = (VT)(pc.M - 1);
            auto stage_of_lane = [&](int a_, int b_) -> VT {         // cost of this lane's stage over (a_, b_]
                const uint8_t *th = thr + ((size_t)lane * T + sp.capt) * R * n1;
                int r = 0;
                for (; r < R - 1; ++r)          // lowest allowed level that fits (the span is feasible, so one does)
                    if (((rc_mask >> r) & 1u) && th[(size_t)r * n1 + b_] <= a_) break;
                const VT *rM = sR + (size_t)sp.mrow * RW * n1;
                if (LINEAR) return (rM[(size_t)r * n1 + b_] - rM[(size_t)r * n1 + a_]) + sp.K;
                return ((rM[b_] - rM[a_]) + tau_term((i64)dc.tau_q[r], rM[n1 + b_] - rM[n1 + a_])) + sp.K;
            };
            // one pass: returns false if no partition respects the limit; else the sum, the largest stage cost of
            // the chosen partition, this lane's span, and in `nxt` the smallest stage cost above the limit
            auto pass = [&](VT limit, VT &psum, VT &pmax, VT &nxt, int &pa, int &pb) -> bool {
                int pbl = 0, pbh = 0;
                VT skipped = vInf;
                for (int i = 1; i <= PP; ++i) {
                    const int src = i - 1;
                    const int mrow = __shfl_sync(0xffffffffu, sp.mrow, src), capt = __shfl_sync(0xffffffffu, sp.capt, src);
                    const VT K = shfl_v(sp.K, src);
                    const int nmin = __shfl_sync(0xffffffffu, sp.nmin, src), nmax = __shfl_sync(0xffffffffu, sp.nmax, src);
                    const int bl = __shfl_sync(0xffffffffu, sp.bl, src), bh = __shfl_sync(0xffffffffu, sp.bh, src);
                    const VT *rM = sR + (size_t)mrow * RW * n1;
                    const VT *prev = i == 1 ? szero : rows2 + (size_t)(i & 1) * n1;
                    VT *cur = rows2 + (size_t)((i - 1) & 1) * n1;
                    uint8_t *chrow = chw + (size_t)(i - 1) * n1;
                    const uint8_t *th = thr + ((size_t)(i - 1) * T + capt) * R * n1;
                    for (int j = bl + lane; j <= bh; j += 32) {
                        VT best = vInf;
                        int arg = 255;
                        int klo = j - nmax; if (klo < pbl) klo = pbl;
                        int khi = j - nmin; if (khi > pbh) khi = pbh;
                        int seg_hi = khi;
                        for (int r = 0; r < R && seg_hi >= klo; ++r) {
                            if (!((rc_mask >> r) & 1u)) continue;
                            int lo = th[(size_t)r * n1 + j];
                            if (lo < klo) lo = klo;
                            if (lo > seg_hi) continue;
                            for (int k = seg_hi; k >= lo; --k) {
                                VT cst;
                                if (LINEAR) cst = (rM[(size_t)r * n1 + j] - rM[(size_t)r * n1 + k]) + K;
                                else cst = ((rM[j] - rM[k]) + tau_term((i64)dc.tau_q[r], rM[n1 + j] - rM[n1 + k])) + K;
                                if (cst > limit) { skipped = cst < skipped ? cst : skipped; continue; }
                                const VT v = prev[k] + cst;
                                if (v <= best && v < vInf) { best = v; arg = k; }
                            }
                            seg_hi = lo - 1;
                        }
                        cur[j] = best;
                        chrow[j] = (uint8_t)arg;
                    }
                    __syncwarp();
                    pbl = bl; pbh = bh;
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) { const VT t = __shfl_xor_sync(0xffffffffu, skipped, o); skipped = t < skipped ? t : skipped; }
                nxt = skipped;
                psum = rows2[(size_t)((PP - 1) & 1) * n1 + N];
                if (!(psum < vInf)) return false;
                int j = N;
                pa = 0; pb = 0;
                for (int i = PP; i >= 1; --i) {
                    const int k = chw[(size_t)(i - 1) * n1 + j];
                    if (lane == i - 1) { pa = k; pb = j; }
                    j = k;
                }
                VT c = lane < PP ? stage_of_lane(pa, pb) : (VT)0;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) { const VT t = __shfl_xor_sync(0xffffffffu, c, o); c = t > c ? t : c; }
                pmax = c;
                __syncwarp();
                return true;
            };
            VT bs, bm, nx;
            pass(bott, bs, bm, nx, ref_a, ref_b);            // always feasible: the min-max partition respects the limit
            if (out.exact) {
                // Sweep.  f_min = the smallest sum without a limit; a partition whose largest stage costs t cannot
                // beat the incumbent V once f_min + (M-1) t >= V.  The first limit that reaches the smallest value wins.
                VT Vbest = bs + M1 * bm;
                VT us, um, unx; int ua, ub;
                pass(vInf - 1, us, um, unx, ua, ub);
                VT t = nx;
                while (t < vInf && us + M1 * t < Vbest) {
                    VT cs, cm, cn; int ca, cb;
                    if (pass(t, cs, cm, cn, ca, cb) && cs + M1 * cm < Vbest) { Vbest = cs + M1 * cm; ref_a = ca; ref_b = cb; }
                    t = cn;
                }
                if (us + M1 * um < Vbest) { ref_a = ua; ref_b = ub; }
            }
        }

        // ---- backtrace, Eq. 4 -----------------------------------------------------------
        VT T_iter = vInf, T_pipe = vInf, T_sync = 0, T_opt = 0;
        int my_n = 0, my_r = 0;
        if (bott < vInf) {
            int a_me = ref_a, b_me = ref_b;
            if (!REFINE) {
                int j = N;
                for (int i = PP; i >= 1; --i) {
                    const int k = chw[(size_t)(i - 1) * n1 + j];
                    if (lane == i - 1) { a_me = k; b_me = j; }
                    j = k;
                }
            }
            VT c_me = 0, sync_me = 0, opt_me = 0;
            if (lane < PP) {
                const uint8_t *th = thr + ((size_t)lane * T + sp.capt) * R * n1;
                int r = 0;
                for (; r < R; ++r)
                    if (((rc_mask >> r) & 1u) && th[(size_t)r * n1 + b_me] <= a_me) break;
                const VT *rM = sR + (size_t)sp.mrow * RW * n1;
                if (LINEAR) c_me = (rM[(size_t)r * n1 + b_me] - rM[(size_t)r * n1 + a_me]) + sp.K;
                else c_me = ((rM[b_me] - rM[a_me]) + tau_term((i64)dc.tau_q[r], rM[n1 + b_me] - rM[n1 + a_me])) + sp.K;
                my_n = b_me - a_me; my_r = r;
                const VT n_moe = (VT)((int)sK[b_me] - (int)sK[a_me]), n_dense = (VT)(b_me - a_me) - n_moe;
                const MaskInfo<VT> &mi_ = minfo[mask - 1];
                sync_me = mi_.slat + n_dense * mi_.sbw[0] + n_moe * mi_.sbw[1];
                opt_me = n_dense * mi_.opt[0] + n_moe * mi_.opt[1];
            }
            VT het_me = 0;                                  // cross-type transfer into this lane's stage (Pruning 3)
            if (dc.eta_q > 0 && lane > 0 && lane < PP && (link & 3) == HAP_CROSS) het_me = sP2P[(link >> 4) & 3][2 + ((link >> 2) & 3)];
            // ... and, when asked for, the dispatch / combine traffic of the MoE layers of a stage that spans device types
            if (dc.eta_q > 0 && lane < PP) het_me += (VT)((int)sK[b_me] - (int)sK[a_me]) * minfo[mask - 1].kxd;
            VT sum = c_me, mxc = c_me;
            for (int o = red0; o > 0; o >>= 1) {          // lanes >= PP hold zeros
                const VT t1 = __shfl_xor_sync(0xffffffffu, sum, o), t2 = __shfl_xor_sync(0xffffffffu, mxc, o);
                const VT t3 = __shfl_xor_sync(0xffffffffu, sync_me, o), t4 = __shfl_xor_sync(0xffffffffu, opt_me, o);
                sum += t1; mxc = t2 > mxc ? t2 : mxc; sync_me = t3 > sync_me ? t3 : sync_me; opt_me = t4 > opt_me ? t4 : opt_me;
            }
            T_pipe = shfl_v(sum + (VT)(pc.M - 1) * mxc, 0);
            T_sync = shfl_v(sync_me, 0); T_opt = shfl_v(opt_me, 0);
            T_iter = T_pipe + T_sync + T_opt;
            if (dc.eta_q > 0) {
                // Pruning 3: cross-type communication per micro-batch above eta x the mean stage time drops the
                // candidate (its bottleneck is still reported)
                for (int o = red0; o > 0; o >>= 1) het_me += __shfl_xor_sync(0xffffffffu, het_me, o);
                const VT het = shfl_v(het_me, 0), ssum = shfl_v(sum, 0);
                if (het * (VT)PP * (VT)1024 > (VT)dc.eta_q * ssum) { T_iter = vInf; T_pipe = vInf; }
            }
        }
        if (SEARCH) {
            n_eval++;
            if (T_iter < vInf) n_feas++;
            if (T_iter < best_cost || (T_iter == best_cost && c < best_index)) {
                best_cost = T_iter; best_index = c;
                if ((out.prune || out.cand_lb) && lane == 0) atomicMin(out.incumbent, (u64)(i64)T_iter);
            }
        } else {
            const u64 o = c - out.first;
            if (lane == 0) {
                if (out.cost) reinterpret_cast<VT *>(out.cost)[o] = T_iter;
                if (out.bottleneck) reinterpret_cast<VT *>(out.bottleneck)[o] = bott;
                if (out.detail) {
                    VT *d = reinterpret_cast<VT *>(out.detail);
                    d[o * 3] = T_pipe; d[o * 3 + 1] = T_sync; d[o * 3 + 2] = T_opt;
                }
            }
            if (out.partition) out.partition[o * HAP_MAX_PP + lane] = (uint8_t)(T_iter < vInf ? my_n : 0);
            if (out.recompute) out.recompute[o * HAP_MAX_PP + lane] = (uint8_t)(T_iter < vInf ? my_r : 0);
        }
        __syncwarp();
      }
      if (lane == 0) s_infeas[wib][rc_pos] = infeasible_here;
      __syncwarp();
    }

    if (out.counters) {
        n_cells = (u64)warp_sum_i64((i64)n_cells);
        if (lane == 0 && n_cells) atomicAdd(out.counters + 4, n_cells);
    }
    if (SEARCH) {
        __shared__ i64 wcost[kDpWarps];
        __shared__ u64 widx[kDpWarps];
        if (lane == 0) {
            wcost[wib] = (i64)best_cost; widx[wib] = best_index;
            if (n_eval) atomicAdd(out.counters + 0, n_eval);
            if (n_feas) atomicAdd(out.counters + 1, n_feas);
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            i64 bc = wcost[0]; u64 bi = widx[0];
            for (int q = 1; q < nwarps; ++q)
                if (wcost[q] < bc || (wcost[q] == bc && widx[q] < bi)) { bc = wcost[q]; bi = widx[q]; }
            out.partial_cost[blockIdx.x] = bc;
            out.partial_index[blockIdx.x] = bi;
        }
    }
}

// ------------------------------------------------------------------------------------------
// joint recurrence over the device state (the DP form printed in Sec. 3.5 / Algorithm 1, min-max objective):
// value[u][t][j] = smallest achievable largest stage cost when the first |u| stages hold the first j layers,
// u[h] of them on device type h, the last one on type t.  One block per configuration; the states of one
// level (= number of stages placed) are spread over the block's warps, lanes run over j; two levels of rows
// live in a per-block slice of a global scratch buffer.  The result for u = "all stages placed", j = N is the
// minimum, over every stage-type sequence, of the bottleneck the per-candidate kernel computes.
// ------------------------------------------------------------------------------------------
struct JointClass {
    int PP, S, lmax;              // stages; number of states; most states of one level
    int cnt[HAP_MAX_TYPES];       // stages of each type
    int stride[HAP_MAX_TYPES];    // mixed-radix strides of the state index
    const int *lvl_off;           // [PP+2] offsets of each level in st_idx
    const int *st_idx;            // [S] state indices ordered by level
    const int *slot;              // [S] rank of a state within its level
    const int *dig;               // [S] in level order: the state's stage counts per type, one byte each
    int *band;                    // [S] in level order: reachable end layers of the state, lo | hi << 8 (filled by the kernel)
};

__host__ __device__ inline size_t joint_smem_bytes(int N, int PP, int T, int R, bool linear)
{
    const size_t n1 = (size_t)N + 1;
    size_t b = (size_t)T * (linear ? (size_t)R : 2) * n1 * 8 + n1 * 16;
    b += ((size_t)PP * T * R * n1 + 15) / 16 * 16;
    b += (n1 + 15) / 16 * 16;
    return b + 32;
}

template <bool LINEAR>
__global__ void __launch_bounds__(256)
joint_dp_kernel(const DevConst dc, const unsigned *pconf_ids, unsigned n_ids, const i64 *c2, const i64 *coef,
                JointClass jc, i64 *scratch, i64 *out)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    typedef i64 VT;
    const int N = dc.N, T = dc.T, R = dc.R, n1 = N + 1, n_rc = dc.n_rc;
    const int wib = threadIdx.x >> 5, lane = threadIdx.x & 31, nwarps = blockDim.x >> 5;
    const int PP = jc.PP;
    const int RW = LINEAR ? R : 2;
    VT *sR = reinterpret_cast<VT *>(smem_raw);
    i64 *sW = reinterpret_cast<i64 *>(sR + (size_t)T * RW * n1);
    i64 *sA = sW + n1;
    uint8_t *thr = reinterpret_cast<uint8_t *>(sA + n1);
    uint8_t *sK = thr + ((size_t)PP * T * R * n1 + 15) / 16 * 16;
    __shared__ MaskInfo<VT> minfo[kMaxMasks];
    __shared__ VT sP2P[HAP_MAX_TYPES][6];
    __shared__ VT szero[1];
    __shared__ int winT[HAP_MAX_TYPES][2];
    const size_t lvl_cells = (size_t)jc.lmax * T * n1;
    i64 *buf0 = scratch + (size_t)blockIdx.x * 2 * lvl_cells, *buf1 = buf0 + lvl_cells;

    for (unsigned w = blockIdx.x; w < n_ids; w += gridDim.x) {
        const unsigned p = pconf_ids[w];
        const hap_pconf pc = dc.pconf[p];
        __syncthreads();                                  // the previous configuration's tables are no longer read
        dp_block_prologue<VT, LINEAR>(dc, pc, p, c2, coef, coef, true, T, RW, 0xffffffffu, nwarps,
                                      sR, sW, sA, thr, sK, minfo, sP2P, szero, winT);
        if (w == blockIdx.x) {
            // End layers a state can have: the stages placed so far and the stages still to place each hold a number
            // of layers inside their type's window (the same for every configuration of the class); a cell outside
            // the band is on no complete partition.  Every block fills the whole table with the same values and
            // reads what it wrote itself.
            for (int pos = threadIdx.x; pos < jc.S; pos += blockDim.x) {
                const int dg = jc.dig[pos];
                int lvl = 0, smin = 0, smax = 0, rmin = 0, rmax = 0;
                for (int h = 0; h < T; ++h) {
                    const int uh = (dg >> (8 * h)) & 255, rh = jc.cnt[h] - uh;
                    lvl += uh;
                    smin += uh * winT[h][0]; smax += uh * winT[h][1];
                    rmin += rh * winT[h][0]; rmax += rh * winT[h][1];
                }
                int bl = smin > N - rmax ? smin : N - rmax, bh = smax < N - rmin ? smax : N - rmin;
                if (bl < lvl) bl = lvl;
                if (bh > N - PP + lvl) bh = N - PP + lvl;
                if (bl > bh || bl < 0) { bl = 255; bh = 0; }
                jc.band[pos] = bl | (bh << 8);
            }
            __threadfence_block();
            __syncthreads();
        }
        for (int rc_idx = 0; rc_idx < n_rc; ++rc_idx) {
            const unsigned rc_mask = dc.rc_masks[rc_idx];
            for (int i = 1; i <= PP; ++i) {
                i64 *cur = (i & 1) ? buf1 : buf0;
                const i64 *prv = (i & 1) ? buf0 : buf1;
                const int l0 = jc.lvl_off[i], l1 = jc.lvl_off[i + 1];
                for (int pr = wib; pr < (l1 - l0) * T; pr += nwarps) {
                    const int sl = pr / T, t = pr - sl * T;
                    const int dg = jc.dig[l0 + sl];
                    const int ut = (dg >> (8 * t)) & 255;
                    i64 *row = cur + ((size_t)sl * T + t) * n1;
                    if (ut == 0) continue;                  // no stage of type t placed: rows of such pairs are never read
                    const int up = jc.st_idx[l0 + sl] - jc.stride[t];
                    const int slot_up = i > 1 ? jc.slot[up] : 0;
                    const int nmin = winT[t][0], nmax = winT[t][1];
                    const uint8_t *th = thr + ((size_t)(i - 1) * T + t) * R * n1;
                    const VT *rM = sR + (size_t)t * RW * n1;
                    const MaskInfo<VT> &mi = minfo[(1 << t) - 1];
                    const VT Kbase = (i == 1 ? mi.kpre : 0) + (i == PP ? mi.kpost : 0);
                    // the q-th stage of its type starts at device q*G of the type's device line
                    const i64 first = (i64)(ut - 1) * pc.G;
                    const int same_cls = ((first - 1) / dc.node_size[t] == first / dc.node_size[t]) ? HAP_INTRA : HAP_INTER;
                    const int bb = jc.band[l0 + sl];
                    const int bl = bb & 255, bh = bb >> 8;
                    // the band of the state before this stage (one stage of type t fewer): its rows hold nothing
                    // outside it, so the splits are clipped to it
                    int pbl = 0, pbh = 0;
                    if (i > 1) {
                        const int pb = jc.band[jc.lvl_off[i - 1] + slot_up];
                        pbl = pb & 255; pbh = pb >> 8;
                    }
                    // four lanes per end layer, one per type of the stage before (T <= 4); the lane's type is fixed
                    const int tp = lane & 3;
                    bool tp_ok = i == 1 ? tp == 0 : tp < T;
                    const VT *prow = szero;
                    VT K = Kbase;
                    if (i > 1 && tp_ok) {
                        const int utp = ((dg >> (8 * tp)) & 255) - (tp == t ? 1 : 0);
                        tp_ok = utp != 0;                      // the prefix contains type tp
                        prow = prv + ((size_t)slot_up * T + tp) * n1;
                        K += tp != t ? sP2P[t][2 + tp] : sP2P[t][same_cls];
                    }
                    const int cells4 = (bh - bl + 1) * 4;
                    for (int base = 0; base < cells4; base += 32) {
                        const int idx = base + lane, j = bl + (idx >> 2);
                        VT best = kInf;
                        if (idx < cells4 && tp_ok) {
                            int kl = j - nmax; if (kl < pbl) kl = pbl;
                            int kh = j - nmin; if (kh > pbh) kh = pbh;
                            int seg_hi = kh;
                            for (int r = 0; r < R && seg_hi >= kl; ++r) {
                                if (!((rc_mask >> r) & 1u)) continue;
                                int lo = th[(size_t)r * n1 + j];
                                if (lo < kl) lo = kl;
                                if (lo > seg_hi) continue;
                                const VT Cj = LINEAR ? rM[(size_t)r * n1 + j] + K : 0;
                                for (int k = seg_hi; k >= lo; --k) {
                                    VT cst;
                                    if (LINEAR) cst = Cj - rM[(size_t)r * n1 + k];
                                    else cst = ((rM[j] - rM[k]) + tau_term((i64)dc.tau_q[r], rM[n1 + j] - rM[n1 + k])) + K;
                                    const VT pv = prow[k];
                                    const VT v = pv > cst ? pv : cst;
                                    best = v < best ? v : best;
                                    // layer times are non-negative: the stage cost only grows as k falls within
                                    // a level, so nothing further down this level can beat the best value
                                    if (cst > best) break;
                                }
                                seg_hi = lo - 1;
                            }
                        }
                        VT o = shfl_i64(best, lane ^ 1); best = o < best ? o : best;
                        o = shfl_i64(best, lane ^ 2); best = o < best ? o : best;
                        if (idx < cells4 && tp == 0) row[j] = best;
                    }
                    // the answer is read at (all stages placed, N): make sure that cell exists
                    if (i == PP && lane == 0 && (N < bl || N > bh)) row[N] = kInf;
                }
                __syncthreads();
            }
            if (threadIdx.x == 0) {
                const i64 *fin = (PP & 1) ? buf1 : buf0;      // level PP has the single state "everything placed"
                VT b = kInf;
                for (int t = 0; t < T; ++t)
                    if (jc.cnt[t] > 0) { const VT v = fin[(size_t)t * n1 + N]; b = v < b ? v : b; }
                out[(size_t)p * n_rc + rc_idx] = b;
            }
            __syncthreads();
        }
    }
}

// ------------------------------------------------------------------------------------------
// argmin: stage 1 reduces a slice per block, stage 2 (one block) reduces the partials
// ------------------------------------------------------------------------------------------
// Lower bounds on T_iter of the candidates of one configuration per block, from the bottlenecks a plain pass left in
// `bound` (in place): any partition of candidate c has a largest stage cost >= B*(c) and a stage-cost sum >= S, the sum
// over layers of the cheapest device type's time, so sum + (M-1) max >= S + (M-1) B*(c); infeasible stays HAP_INF.
__global__ void cand_bound_kernel(const DevConst dc, const i64 *__restrict__ lb_sum, i64 *bound, u64 first, u64 count)
{
    const u64 p = blockIdx.x;
    const hap_pconf pc = dc.pconf[p];
    const u64 c0 = pc.offset, c1 = c0 + pc.nmap * (u64)dc.n_rc;
    const u64 a = c0 > first ? c0 : first, b = c1 < first + count ? c1 : first + count;
    const i64 S = lb_sum[p], m1 = (i64)pc.M - 1;
    for (u64 c = a + threadIdx.x; c < b; c += blockDim.x) {
        const i64 bott = bound[c];
        bound[c] = bott >= kInf ? kInf : S + m1 * bott;
    }
}

// an index relative to a range start becomes a global candidate index (negative: none, stays negative)
__global__ void offset_index_kernel(i64 *index, i64 first)
{
    if (threadIdx.x == 0 && blockIdx.x == 0 && *index >= 0) *index += first;
}

// the incumbent of a search starts at the cost of one evaluated candidate
// (index < 0: no candidate was evaluated, the incumbent stays at +INF)
__global__ void set_incumbent_kernel(u64 *incumbent, const i64 *cost, const i64 *index)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) { const i64 c = *index < 0 ? kInf : *cost; *incumbent = c < kInf ? (u64)c : (u64)kInf; }
}

// "no candidate" into partial-minimum slots that no block of the pass writes
__global__ void fill_partials_kernel(i64 *pcost, u64 *pindex, unsigned n)
{
    const unsigned q = blockIdx.x * blockDim.x + threadIdx.x;
    if (q < n) { pcost[q] = kInf; pindex[q] = ~0ull; }
}

__global__ void __launch_bounds__(256)
argmin_partial_kernel(const i64 *cost, u64 count, i64 *pcost, u64 *pindex, i64 init)
{
    // `init` is the value reported when nothing is smaller: HAP_INF for integer costs, INT64_MAX when the
    // array holds the bit patterns of non-negative doubles (which order like the doubles themselves)
    asm volatile("griddepcontrol.launch_dependents;");      // the one-block second stage may be brought up meanwhile
    i64 bc = init; u64 bi = ~0ull;
    for (u64 i = (u64)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (u64)gridDim.x * blockDim.x) {
        const i64 v = cost[i];
        if (v < bc) { bc = v; bi = i; }      // ascending i per thread: strict keeps the lowest index
    }
    warp_argmin(bc, bi);
    __shared__ i64 sc[8]; __shared__ u64 si[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { sc[w] = bc; si[w] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int q = 1; q < 8; ++q) if (sc[q] < bc || (sc[q] == bc && si[q] < bi)) { bc = sc[q]; bi = si[q]; }
        pcost[blockIdx.x] = bc; pindex[blockIdx.x] = bi;
    }
}

__global__ void __launch_bounds__(256)
argmin_final_kernel(const i64 *pcost, const u64 *pindex, u64 n, i64 *out2, i64 init, const PlanSlot *plans = nullptr,
                    i64 *w_vals = nullptr, uint8_t *w_part = nullptr, uint8_t *w_rec = nullptr)
{
    // launched as a programmatic dependent of the first stage where it follows one directly: the partials are
    // complete and visible after this wait (a no-op in an ordinary launch)
    asm volatile("griddepcontrol.wait;" ::: "memory");
    i64 bc = init; u64 bi = ~0ull;
    for (u64 i = threadIdx.x; i < n; i += blockDim.x) {
        const i64 v = pcost[i]; const u64 ix = pindex[i];
        if (v < bc || (v == bc && ix < bi)) { bc = v; bi = ix; }
    }
    warp_argmin(bc, bi);
    __shared__ i64 sc[8]; __shared__ u64 si[8];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { sc[w] = bc; si[w] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int q = 1; q < 8; ++q) if (sc[q] < bc || (sc[q] == bc && si[q] < bi)) { bc = sc[q]; bi = si[q]; }
        out2[0] = bc; out2[1] = (i64)bi;
        sc[0] = bc; si[0] = bi;
        if (plans) w_vals[0] = init;             // (a winner whose plan is not found below shows as a cost that differs)
    }
    if (!plans) return;
    // the block that reported the minimum also left the candidate's plan: copy it beside the minimum
    // (w_vals: cost, bottleneck, T_pipe, T_sync, T_opt)
    __syncthreads();
    bc = sc[0]; bi = si[0];
    if (!(bc < init)) return;
    for (u64 i = threadIdx.x; i < n; i += blockDim.x)
        if (pindex[i] == bi && pcost[i] == bc) {
            const PlanSlot ps = plans[i];
            w_vals[0] = bc; w_vals[1] = ps.bott; w_vals[2] = ps.T_pipe; w_vals[3] = ps.T_sync; w_vals[4] = ps.T_opt;
            for (int q = 0; q < HAP_MAX_PP; ++q) { w_part[q] = q < ps.PP ? ps.n[q] : 0; w_rec[q] = q < ps.PP ? ps.r[q] : 0; }
        }
}

}  // namespace hap

// Prefix-tree form of the min-max pipeline recurrence (sm_100a).
//
// The DP row of stage d of a candidate depends only on the candidate's stages 1..d (their device
// types, boundary links and load-balance windows), the configuration and the recomputation policy.
// All mappings of a PP class therefore form a prefix tree whose nodes are distinct stage prefixes;
// the tree, the band of reachable end layers of every node and the flat list of (node, end layer)
// cells of every depth depend on the class alone and are built once on the host.
//
//   trie_dp_kernel   one block per (configuration, part of the tree).  After the block prologue (stage rows, memory
//                    thresholds) the block walks the tree depth by depth: one thread per cell
//                    (node, j) runs the split loop over k against the parent node's row; rows of two
//                    consecutive depths live in shared memory, split choices of all depths as bytes.
//                    Then one thread per mapping evaluates the last stage's single cell (PP, N), walks
//                    the split choices back through the node's ancestors and assembles Eq. 4.
//                    Integer and fp64 mode, level-combined rows only (recomputation factors that are
//                    multiples of 1024); DP tables and the refinement modes run in pipeline_dp_kernel.
#pragma once
#include "hap_device.cuh"

namespace hap {

struct TrieNode {            // a distinct prefix of stages 1..d, d < PP               (16 bytes)
    u32 rowoff;              // first cell of the node's row within its depth
    u32 prowoff;             // the same for the parent node (depth d-1)
    uint8_t mask, link;      // stage d: device types, boundary link into the stage
    uint8_t nmin, nmax;      // stage d: load-balance window on the layer count
    uint8_t bl, bh;          // band of end layers of stage d (union over the mappings below the node)
    uint8_t pbl, pbh;        // the parent's band (stage 0: {0})
};

struct TrieLeaf {            // one mapping: its last stage                              (16 bytes)
    u32 prowoff;             // row of the node of depth PP-1
    uint16_t parent;         // that node's index within its depth
    uint8_t mask, link, nmin, nmax, pbl, pbh;
    uint8_t dead;            // the windows of this mapping cannot add up to N
    uint8_t capt;            // device type whose memory binds the stage
    uint8_t pad[2];
};

// One cell (node, end layer j) of a depth d < PP: everything its split loop needs, in 16 bytes.
//   x = (row origin of the parent in the previous depth's buffer, i.e. prowoff - pbl, + 256) | kidx << 26
//       kidx: entry of the block's table of stage constants (depth 1: pre-work of the stage's types;
//       deeper: p2p transfer by receiving type and link class), filled from the decode of each pass
//   y = j | klo << 8 | khi << 16          (klo..khi: window of the stage within the parent's band)
//   z = index of the cell's level-0 memory threshold in the block's threshold table
//   w = element offset of the level-0 time row of the stage's type mask
typedef uint4 TrieCell;

struct TrieMeta {
    const TrieNode *nodes;          // grouped by depth
    const uint16_t *parent;         // per node: index of its parent within depth d-1
    const TrieCell *cells;          // grouped by depth
    const TrieLeaf *leaves;         // [nmap]
    u32 node_lo[HAP_MAX_PP + 1];    // nodes of depth d: [node_lo[d], node_lo[d+1]), d = 1..PP-1
    u32 cell_lo[HAP_MAX_PP + 1];    // cells of depth d: [cell_lo[d], cell_lo[d+1])
    uint8_t jlo[HAP_MAX_PP + 1], jhi[HAP_MAX_PP + 1];   // end layers that occur at depth d (depth PP: N)
    uint8_t wmax[HAP_MAX_PP + 1];   // widest window of a stage at depth d
    uint8_t tmask[HAP_MAX_PP + 1];  // device types whose memory binds some stage of depth d
    uint8_t kmin[HAP_MAX_PP + 1], kmax[HAP_MAX_PP + 1];   // smallest / largest split any cell of depth d looks at
    uint8_t mrow_of[16];            // type mask -> its row group in the block's time rows (255: no stage has this mask)
    uint8_t mask_of_row[16];        // the inverse
    int n_mrows;
    u32 buf_cells[2];               // largest row storage of an even / odd depth, in cells
    u32 nmap, m_lo;                 // the tree covers mappings [m_lo, m_lo + nmap) of the class
    int PP, band_max;               // band_max: most end layers of any depth
    int thr_w;                      // entries per row of the threshold table: band_max, or 1 when every depth is flat
    uint8_t flat[HAP_MAX_PP + 1];   // depth d sees spans of one layer kind only: its threshold rows hold one entry (column 0)
    uint8_t all_flat;               // every depth is
    uint8_t pad_flat[2];
};

constexpr int kTrieKtab = 16 + HAP_MAX_TYPES * 6;    // stage constants: [0,16) pre-work by row group, then p2p [type][6]

__host__ __device__ inline size_t trie_smem_bytes(int N, int PP, int T, int R, int n_mrows, int thr_w, u32 buf_even, u32 buf_odd, u32 cells,
                                                  u32 n_nodes)
{
    const size_t n1 = (size_t)N + 1;
    size_t b = (((size_t)n_mrows * R + 2) * n1 * 8 + 15) / 16 * 16;      // time rows, weight and activation byte rows
    b += ((size_t)PP * T * R * thr_w + 15) / 16 * 16;                     // memory thresholds
    b += (n1 + 15) / 16 * 16;                                              // MoE prefix counts
    b += (size_t)T * N * 16;                                               // staged layer times of the configuration
    b += (size_t)kTrieKtab * 8;
    b += ((size_t)buf_even + buf_odd) * 8;
    b += ((size_t)cells + 15) / 16 * 16;
    b += (size_t)n_nodes * 16 + ((size_t)n_nodes * 2 + 15) / 16 * 16;      // node records and parent indices
    return b + 32;
}

struct TrieRowMap { uint8_t mrow_of[16]; };

template <typename T> struct IsF64 { static constexpr bool value = false; };
template <> struct IsF64<double> { static constexpr bool value = true; };

// Copies what the decode of this pass produced into the tree: node n of depth d takes the stage bytes (device
// types, boundary link) of stage d of the first mapping below it, every cell of the node the index of the stage
// constant that follows from them, leaf m the last stage of mapping m.
__device__ __forceinline__ void trie_gather_one(const uint8_t *__restrict__ maptab, int PP, u32 n_nodes, u32 n_cells, u32 nmap, u32 m_lo,
                                                const u32 *__restrict__ first_leaf, const uint8_t *__restrict__ depth,
                                                const u32 *__restrict__ cell_gnode, const TrieRowMap &rm,
                                                TrieNode *nodes, TrieCell *cells, TrieLeaf *leaves, u32 g)
{
    if (g < n_nodes) {
        const uint8_t *src = maptab + ((u64)first_leaf[g] * PP + (depth[g] - 1)) * 2;
        nodes[g].mask = src[0]; nodes[g].link = src[1];
    } else if (g < n_nodes + n_cells) {
        const u32 c = g - n_nodes, nd = cell_gnode[c];
        if (!HAP_CHECK_OK(8, nd < n_nodes)) return;
        const int d = depth[nd];
        if (!HAP_CHECK_OK(8, d >= 1 && d < PP)) return;
        const uint8_t *src = maptab + ((u64)first_leaf[nd] * PP + (d - 1)) * 2;
        const int mask = src[0] & 15, link = src[1];
        const int cls = link & 3, ha = (link >> 2) & 3, hb = (link >> 4) & 3;
        const u32 kidx = d == 1 ? rm.mrow_of[mask] : 16 + hb * 6 + (cls == HAP_CROSS ? 2 + ha : cls);
        u32 *x = reinterpret_cast<u32 *>(cells + c);
        *x = (*x & 0x03ffffffu) | (kidx << 26);
    } else if (g < n_nodes + n_cells + nmap) {
        const u32 m = g - n_nodes - n_cells;
        const uint8_t *src = maptab + ((u64)(m_lo + m) * PP + (PP - 1)) * 2;
        leaves[m].mask = src[0]; leaves[m].link = src[1];
    }
}

__global__ void trie_gather_kernel(const uint8_t *__restrict__ maptab, int PP, u32 n_nodes, u32 n_cells, u32 nmap, u32 m_lo,
                                   const u32 *__restrict__ first_leaf, const uint8_t *__restrict__ depth,
                                   const u32 *__restrict__ cell_gnode, const TrieRowMap rm,
                                   TrieNode *nodes, TrieCell *cells, TrieLeaf *leaves)
{
    trie_gather_one(maptab, PP, n_nodes, n_cells, nmap, m_lo, first_leaf, depth, cell_gnode, rm, nodes, cells, leaves,
                    blockIdx.x * blockDim.x + threadIdx.x);
}

// The same for every part of every class's tree in one launch: part q owns blocks [blk_lo, blk_lo + blocks) of 256
// threads (the job list lives in device memory: it is fixed once the trees are built).
struct GatherJob {
    const u32 *first_leaf, *gnode;
    const uint8_t *depth;
    TrieNode *nodes;
    TrieCell *cells;
    TrieLeaf *leaves;
    u64 tab_off;                 // byte offset of the class's decoded-mapping table
    u32 n_nodes, n_cells, nmap, m_lo, blk_lo;
    int PP;
    TrieRowMap rm;
};

__global__ void __launch_bounds__(256) trie_gather_all_kernel(const GatherJob *__restrict__ jobs, int n_jobs, const uint8_t *__restrict__ tab_base)
{
    int q = 0;
    while (q + 1 < n_jobs && blockIdx.x >= jobs[q + 1].blk_lo) ++q;
    const GatherJob &jb = jobs[q];
    trie_gather_one(tab_base + jb.tab_off, jb.PP, jb.n_nodes, jb.n_cells, jb.nmap, jb.m_lo, jb.first_leaf, jb.depth, jb.gnode, jb.rm,
                    jb.nodes, jb.cells, jb.leaves, (blockIdx.x - jb.blk_lo) * blockDim.x + threadIdx.x);
}

// shared-memory accesses by 32-bit address (the split loop walks two rows with plain address decrements)
__device__ __forceinline__ u32 smem_u32(const void *p) { return (u32)__cvta_generic_to_shared(p); }
#ifdef HAP_CHECKED
__device__ __forceinline__ bool smem_addr_ok(u32 a, u32 bytes)
{
    // the dynamic part lies behind the static variables of the kernel: nothing is addressable past its end
    extern __shared__ __align__(16) unsigned char dyn_smem_base[];
    u32 dyn;
    asm volatile("mov.u32 %0, %%dynamic_smem_size;" : "=r"(dyn));
    return HAP_CHECK_OK(0, a % bytes == 0 && a + bytes <= smem_u32(dyn_smem_base) + dyn);
}
#else
__device__ __forceinline__ bool smem_addr_ok(u32, u32) { return true; }
#endif
template <int OFF> __device__ __forceinline__ i64 lds_i64(u32 a)
{
    if (!smem_addr_ok(a + (u32)OFF, 8)) return 0;
    i64 v;
    asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(v) : "r"(a), "n"(OFF));
    return v;
}
template <int OFF> __device__ __forceinline__ double lds_f64(u32 a)
{
    if (!smem_addr_ok(a + (u32)OFF, 8)) return 0.0;
    double v;
    asm volatile("ld.shared.f64 %0, [%1+%2];" : "=d"(v) : "r"(a), "n"(OFF));
    return v;
}
__device__ __forceinline__ int lds_u8(u32 a)
{
    if (!smem_addr_ok(a, 1)) return 0;
    u32 v;
    asm volatile("ld.shared.u8 %0, [%1];" : "=r"(v) : "r"(a));
    return (int)v;
}

// Layer times of the configuration into shared memory, computed from the profiled tables and the per-(configuration,
// type) constants of Eq. 2: one thread per (type, layer), with the arithmetic of layer_cost_kernel (same function,
// same bits).  No barrier.
template <typename VT>
__device__ __forceinline__ void trie_compute_costs(const double2 *tab, size_t stride_h, int N, int T, double kappa, u64 kb0, u64 kb1,
                                                u64 kb2, u64 kb3, const TypeConst *tcp, u64 *range_flag, VT *sC)
{
    bool bad = false;
    for (int q = threadIdx.x; q < T * N; q += blockDim.x) {
        const int h = q / N, l = q - h * N;
        const u64 kb = l < 64 ? kb0 : l < 128 ? kb1 : l < 192 ? kb2 : kb3;
        const bool dense = ((kb >> (l & 63)) & 1ull) == (u64)HAP_DENSE;
        const double2 *tp = tab + (size_t)h * stride_h + (size_t)l * 2;
        const double2 ta = __ldg(tp);
        const double2 tf = dense ? make_double2(0.0, 0.0) : __ldg(tp + 1);
        double cf, cb;
        layer_cost_pair(reinterpret_cast<const double2 *>(tcp + h), ta, tf, dense, kappa, cf, cb);
        bad |= !(cf < 6.8719e10) | !(cb < 6.8719e10);                                 // 2^36 ns per layer
        if (IsF64<VT>::value) { sC[(size_t)q * 2] = (VT)cf; sC[(size_t)q * 2 + 1] = (VT)cb; }
        else { sC[(size_t)q * 2] = (VT)__double2ll_rn(cf); sC[(size_t)q * 2 + 1] = (VT)__double2ll_rn(cb); }
    }
    if (bad && range_flag) atomicOr(range_flag, 1ull);
}

// The same from the layer-cost array of a preceding launch, or computed here when the pass hands the constants instead.
template <typename VT>
__device__ __forceinline__ void trie_stage_costs(const DevConst &dc, const hap_pconf &pc, unsigned p_index, const VT *c2,
                                                 const TypeConst *tcg, u64 *range_flag, VT *sC)
{
    const int N = dc.N, T = dc.T, tid = threadIdx.x, nthreads = blockDim.x;
    if (!tcg) {
        const longlong2 *src = reinterpret_cast<const longlong2 *>(c2 + (size_t)p_index * T * N * 2);
        longlong2 *dst = reinterpret_cast<longlong2 *>(sC);
        for (int q = tid; q < T * N; q += nthreads) dst[q] = src[q];
        return;
    }
    const size_t row = ((size_t)pc.itp * dc.ncp + pc.icp) * dc.nmb + pc.ib;            // the same table row for every type
    const size_t stride_h = (size_t)dc.ntp * dc.ncp * dc.nmb * N * 2;                   // 16-byte pairs between device types
    trie_compute_costs<VT>(reinterpret_cast<const double2 *>(dc.tab4) + row * N * 2, stride_h, N, T, dc.kappa, dc.kindbits[0],
                           dc.kindbits[1], dc.kindbits[2], dc.kindbits[3], tcg + (size_t)p_index * T, range_flag, sC);
}

// Block prologue, part 1: the weight and activation byte prefixes, MoE prefix counts, per-mask stage info, p2p
// coefficients, the table of stage constants and a copy of the tree's node records.
template <typename VT>
__device__ __forceinline__ void trie_prologue_rows(
    const DevConst &dc, const TrieMeta &tm, unsigned p_index, const i64 *coef, const VT *coefv,
    i64 *sW, i64 *sA, uint8_t *sK, double *sKtab, TrieNode *sNodes, uint16_t *sParent,
    MaskInfo<VT> *minfo, VT (*sP2P)[6], double *szero)
{
    const int N = dc.N, T = dc.T;
    const int tid = threadIdx.x, nthreads = blockDim.x, nwarps = nthreads >> 5, wib = tid >> 5, lane = tid & 31;
    const int nmask = (1 << T) - 1;
    const i64 *cfp = coef + (size_t)p_index * T * HAP_NCOEF;         // byte coefficients: integers in both modes
    const VT *cvp = coefv + (size_t)p_index * T * HAP_NCOEF;         // time coefficients
    for (int l = tid; l <= N; l += nthreads) sK[l] = (uint8_t)moe_before(dc, l);
    if (tid < nmask) {
        const int mk = tid + 1;
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
        minfo[tid] = mi;
        if (tm.mrow_of[mk] != 255) sKtab[tm.mrow_of[mk]] = (double)mi.kpre;
    }
    if (tid >= 32 && tid < 32 + T * 6) {
        const int q = tid - 32, h = q / 6, e = q % 6;
        const VT v = cvp[h * HAP_NCOEF + HAP_KP2P_INTRA + e];       // intra, inter, cross[0..3] are consecutive columns
        sP2P[h][e] = v;
        sKtab[16 + q] = (double)v;
    }
    if (tid == 0) szero[0] = 0.0;
    // the tree's node records (for the walk back through a mapping's ancestors)
    {
        const uint4 *src = reinterpret_cast<const uint4 *>(tm.nodes);
        uint4 *dst = reinterpret_cast<uint4 *>(sNodes);
        const u32 n_nodes = tm.node_lo[tm.PP];
        for (u32 q = tid; q < n_nodes; q += nthreads) { dst[q] = src[q]; sParent[q] = tm.parent[q]; }
    }
    // weight and activation byte prefixes: one warp, inclusive scans over chunks of 32 layers
    if (wib == nwarps - 1) {
        i64 runA = 0, runB = 0;
        for (int base = 0; base < N; base += 32) {
            const int l = base + lane;
            i64 vA = 0, vB = 0;
            if (l < N) { const int kd = layer_kind(dc, l); vA = cfp[HAP_MW + kd]; vB = cfp[HAP_MA + kd]; }
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const i64 tA = __shfl_up_sync(0xffffffffu, vA, o), tB = __shfl_up_sync(0xffffffffu, vB, o);
                if (lane >= o) { vA += tA; vB += tB; }
            }
            vA += runA; vB += runB;
            if (l < N) { sW[l + 1] = vA; sA[l + 1] = vB; }
            runA = shfl_i64(vA, 31); runB = shfl_i64(vB, 31);
        }
        if (lane == 0) { sW[0] = 0; sA[0] = 0; }
    }
    __syncthreads();
}

// Block prologue, part 2 (configurations that can be feasible): per type mask that occurs in the class the prefix
// rows of the stage time at every recomputation level, fwd+bwd + (tau_r/1024) fwd; one warp per mask, inclusive
// warp scans over chunks of 32 layers.  No barrier: the threshold sweep that follows ends with one.
template <typename VT>
__device__ __forceinline__ void trie_prologue_time_rows(const DevConst &dc, const TrieMeta &tm, const VT *sC, double *sR)
{
    const int N = dc.N, T = dc.T, R = dc.R, n1 = N + 1;
    const int nwarps = blockDim.x >> 5, wib = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int mr = wib; mr < tm.n_mrows; mr += nwarps) {
        const int mk = tm.mask_of_row[mr];
        VT runA = 0, runB = 0;
        for (int base = 0; base < N; base += 32) {
            const int l = base + lane;
            VT vA = 0, vB = 0;                                       // fwd+bwd, fwd
            if (l < N) {
                VT F = 0, B = 0;
                for (int h = 0; h < T; ++h)
                    if (mk >> h & 1) {
                        const VT qx = sC[((size_t)h * N + l) * 2], qy = sC[((size_t)h * N + l) * 2 + 1];
                        F = qx > F ? qx : F;
                        B = qy > B ? qy : B;
                    }
                vA = F + B; vB = F;
            }
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const VT tA = __shfl_up_sync(0xffffffffu, vA, o), tB = __shfl_up_sync(0xffffffffu, vB, o);
                if (lane >= o) { vA += tA; vB += tB; }
            }
            vA += runA; vB += runB;
            if (l < N) for (int r = 0; r < R; ++r) sR[((size_t)mr * R + r) * n1 + l + 1] = (double)(vA + (VT)(dc.tau_q[r] >> 10) * vB);
            runA = shfl_v(vA, 31); runB = shfl_v(vB, 31);
        }
        if (lane == 0) for (int r = 0; r < R; ++r) sR[((size_t)mr * R + r) * n1] = 0.0;
    }
}

// index of the memory threshold of (stage d, capacity type t, level r, end layer j) in the block's table
__device__ __forceinline__ u32 trie_thr_index(const TrieMeta &tm, int T, int R, int d, int t, int r, int j)
{
    return (u32)((((d - 1) * T + t) * R + r) * tm.thr_w + ((tm.thr_w == 1 || tm.flat[d]) ? 0 : j - (int)tm.jlo[d]));
}

// Block prologue, part 3: threshold table: for stage d on a device of type t at level r, the length of the longest
// span ending at layer j that fits (among the splits a cell of depth d can look at; 0: none), only for the end
// layers, device types and levels that occur at depth d; one entry per row at the depths whose spans are of one layer
// kind.  Feasibility is monotone in the span, so for the other depths a thread sweeps the end layers of a row with a
// split pointer that only moves forward.
__device__ __forceinline__ void trie_prologue_thr(
    const DevConst &dc, const hap_pconf &pc, const TrieMeta &tm, unsigned p_index, const i64 *coef, unsigned levels,
    const i64 *sW, const i64 *sA, uint8_t *thr, const uint8_t *sK)
{
    const int T = dc.T, R = dc.R, PP = pc.PP;
    const i64 *cfp = coef + (size_t)p_index * T * HAP_NCOEF;
    const i64 mx = cfp[HAP_MX], mpre = cfp[HAP_MPRE], mpost = cfp[HAP_MPOST];
    {
        // Flat depths (every span a cell of the depth can look at lies behind the last change of layer kind): the
        // memory of a span depends on its length alone, so a row is one number, the longest span that fits (a
        // search over the lengths a window of this depth allows, on spans that end at the last layer).
        const int N = dc.N, rows = PP * T * R;
        const int len_cap = N - dc.kind_uniform_from;
        for (int q = threadIdx.x; q < rows; q += blockDim.x) {
            const int r = q % R, t = (q / R) % T, d = q / (R * T) + 1;
            if (!tm.flat[d]) continue;
            int fit = 0;
            if (((levels >> r) & 1u) && ((tm.tmask[d] >> t) & 1u)) {
                const i64 extra = (d == 1 ? mpre : 0) + (d == PP ? mpost : 0);
                const int inflight = PP - d + 1;
                const i64 mstore = pc.M < inflight ? pc.M : inflight;
                int lo = 0, hi = tm.wmax[d] < len_cap ? tm.wmax[d] : len_cap;   // invariant: lengths <= lo fit (0: trivially), lengths > hi do not
                while (lo < hi) {
                    const int mid = (lo + hi + 1) >> 1;
                    if (span_fits(sW, sA, sK, extra, mx, mstore, dc.cap_eff[t], dc.xi_q[r], N - mid, N)) lo = mid; else hi = mid - 1;
                }
                fit = lo;
            }
            thr[(size_t)q * tm.thr_w] = (uint8_t)fit;
        }
        if (tm.all_flat) { __syncthreads(); return; }
    }
    // end layers per thread: a whole row (fewest evaluations: the pointer never restarts) when the rows alone keep
    // half the block busy, segments of eight otherwise
    const int kSeg = PP * T * R * 2 >= (int)blockDim.x ? 32 : 8;
    const int nseg = (tm.band_max + kSeg - 1) / kSeg;
    const int total = PP * T * R * nseg;
    for (int e = threadIdx.x; e < total; e += blockDim.x) {
        const int seg = e % nseg, q = e / nseg;
        const int r = q % R, t = (q / R) % T, d = q / (R * T) + 1;
        if (tm.flat[d] || !((levels >> r) & 1u) || !((tm.tmask[d] >> t) & 1u)) continue;
        const int j0 = tm.jlo[d] + seg * kSeg;
        int j1 = j0 + kSeg - 1; if (j1 > tm.jhi[d]) j1 = tm.jhi[d];
        if (j0 > j1) continue;
        const i64 extra = (d == 1 ? mpre : 0) + (d == PP ? mpost : 0);
        const int inflight = PP - d + 1;
        const i64 mstore = pc.M < inflight ? pc.M : inflight;
        const i64 cap = dc.cap_eff[t], xi = dc.xi_q[r];
        const int wmax = tm.wmax[d];
        uint8_t *row = thr + (size_t)q * tm.band_max - tm.jlo[d];
        int k = tm.kmin[d];
        const int kmax = tm.kmax[d];
        for (int j = j0; j <= j1; ++j) {
            if (k < j - wmax) k = j - wmax;
            const int kcap = kmax < j - 1 ? kmax : j - 1;           // no cell looks at a split beyond this
            // span (k, j] fits: weights + extra (+ MoE buffers if it holds an MoE layer) + xi * stored activations / 1024
            const i64 Wj = sW[j] + extra, Aj = sA[j];
            const int Kj = sK[j];
            while (k <= kcap) {
                const i64 Wb = (Wj - sW[k]) + (Kj != sK[k] ? mx : 0);
                const i64 A = mstore * (Aj - sA[k]);
                if (Wb + ((xi * A) >> 10) <= cap) break;
                ++k;
            }
            row[j] = (uint8_t)(k <= kcap ? j - k : 0);              // the longest span ending at j that fits (0: none)
        }
    }
    __syncthreads();
}

// VT: i64 (times rounded to integer ns: every operation below is exact) or double (fp64 mode: unrounded times,
// the same steps in floating point; not instantiated for SEARCH).
// COUNT: also count the splits the block evaluates (after its early exits) into out.counters[4]; the counting costs a
// few percent, so only passes of a problem created with HAP_OPT_COUNT_SPLITS run this form.
template <bool SEARCH, int MAXT, int MINB, typename VT = i64, bool COUNT = false>
__global__ void __launch_bounds__(MAXT, MINB)
trie_dp_kernel(const DevConst dc, const u32 *plist, unsigned n_active, const VT *c2, const i64 *coef, const VT *coefv,
               const TrieMeta *metas, int n_parts, DpOut out)
{
    constexpr bool F64 = IsF64<VT>::value;
    static_assert(!(SEARCH && F64), "the fp64 search reduces a cost array; the tree kernel only fills it");
    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ MaskInfo<VT> minfo[kMaxMasks];
    __shared__ VT sP2P[HAP_MAX_TYPES][6];
    __shared__ double szero[1];
    __shared__ i64 wcost[32];
    __shared__ u64 widx[32];
    __shared__ int s_skip;
    __shared__ u64 s_clo;               // first candidate of the block
    __shared__ int s_whole;             // every candidate of the block is wanted
    __shared__ unsigned long long s_lb;

    const int tid = threadIdx.x, nthreads = blockDim.x, nwarps = nthreads >> 5, lane = tid & 31, wib = tid >> 5;
    if (blockIdx.x >= n_active) {
        if (SEARCH && tid == 0) { out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull; }
        return;
    }
    // block -> (configuration, part of the class's tree); the part's description goes to shared memory
    __shared__ TrieMeta tm;
    {
        const u32 *src = reinterpret_cast<const u32 *>(metas + blockIdx.x % (unsigned)n_parts);
        u32 *dst = reinterpret_cast<u32 *>(&tm);
        for (int q = tid; q < (int)(sizeof(TrieMeta) / 4); q += nthreads) dst[q] = src[q];
    }
    __syncthreads();
    const u32 p = plist[blockIdx.x / (unsigned)n_parts];
    if (!HAP_CHECK_OK(7, (u64)p < dc.n_pconf)) return;
    const hap_pconf pc = dc.pconf[p];
    const int N = dc.N, T = dc.T, R = dc.R, n1 = N + 1, PP = pc.PP, n_rc = dc.n_rc, bw = tm.thr_w;
    const u64 c_lo = pc.offset + (u64)tm.m_lo * n_rc, c_hi = c_lo + (u64)tm.nmap * n_rc;   // candidates of this block
    const u64 w_lo = out.first, w_hi = out.first + out.count;                  // candidates that are wanted
    // (the phases after the prologue read the block's range from shared memory: fewer live registers in the split loop)
    if (tid == 0) { s_clo = c_lo; s_whole = c_lo >= w_lo && c_hi <= w_hi; }
    // how many wanted candidates this block stands for
    auto block_candidates = [&]() -> u64 {
        const u64 a = c_lo > w_lo ? c_lo : w_lo, b = c_hi < w_hi ? c_hi : w_hi;
        return b > a ? b - a : 0;
    };
    if (c_hi <= w_lo || c_lo >= w_hi) {
        if (SEARCH && tid == 0) { out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull; }
        return;
    }
    // T_iter >= S + (M-1) ceil(S / PP) with S the configuration's lower bound on the summed stage time (the sum over
    // layers of the cheapest device type's time); one thread reads the moving incumbent and the block follows that
    // reading as a whole.  S comes from the layer-cost kernel, or from this block's own layer times further down.
    if (SEARCH && out.prune && !out.tcg) {
        if (tid == 0) {
            const i64 S = out.lb_sum[p];
            const i64 lb = S + (i64)(pc.M - 1) * ((S + PP - 1) / PP);
            const u64 inc = *reinterpret_cast<volatile const u64 *>(out.incumbent);
            s_skip = (u64)lb > inc;
            if (s_skip) {
                out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull;
                atomicAdd(out.counters + 2, block_candidates());
            }
        }
        __syncthreads();
        if (s_skip) return;
    }

    // shared memory: time rows | weight bytes | activation bytes | thresholds | MoE counts | staged layer times |
    //                stage constants | rows of the even depths | rows of the odd depths | split choices
    double *sR = reinterpret_cast<double *>(smem_raw);
    i64 *sW = reinterpret_cast<i64 *>(sR + (size_t)tm.n_mrows * R * n1);
    i64 *sA = sW + n1;
    const size_t thr_off = (((size_t)tm.n_mrows * R + 2) * n1 * 8 + 15) / 16 * 16;
    uint8_t *thr = smem_raw + thr_off;
    const size_t thr_bytes = ((size_t)PP * T * R * bw + 15) / 16 * 16;
    uint8_t *sK = thr + thr_bytes;
    VT *sC = reinterpret_cast<VT *>(sK + ((size_t)n1 + 15) / 16 * 16);        // [T][N][2], 16-byte aligned
    double *sKtab = reinterpret_cast<double *>(sC + (size_t)T * N * 2);
    double *bufE = sKtab + kTrieKtab;
    double *bufO = bufE + tm.buf_cells[0];
    uint8_t *ch = reinterpret_cast<uint8_t *>(bufO + tm.buf_cells[1]);
    TrieNode *sNodes = reinterpret_cast<TrieNode *>(ch + ((size_t)tm.cell_lo[PP] + 15) / 16 * 16);
    uint16_t *sParent = reinterpret_cast<uint16_t *>(sNodes + tm.node_lo[PP]);

    const i64 *cfp = coef + (size_t)p * T * HAP_NCOEF;

    // writes "infeasible" for candidate c (non-search mode)
    const VT vInf = ValInf<VT>::get();
    auto put_infeasible = [&](u64 c) {
        const u64 o = c - out.first;
        if (out.cost) reinterpret_cast<VT *>(out.cost)[o] = vInf;
        if (out.bottleneck) reinterpret_cast<VT *>(out.bottleneck)[o] = vInf;
        if (out.detail) { VT *dt = reinterpret_cast<VT *>(out.detail); dt[o * 3] = vInf; dt[o * 3 + 1] = 0; dt[o * 3 + 2] = 0; }
        if (out.partition) for (int s = 0; s < HAP_MAX_PP; ++s) out.partition[o * HAP_MAX_PP + s] = 0;
        if (out.recompute) for (int s = 0; s < HAP_MAX_PP; ++s) out.recompute[o * HAP_MAX_PP + s] = 0;
    };

    i64 best_cost = kInf;
    u32 best_local = ~0u;               // the best candidate's offset from the block's first candidate
    u32 n_eval = 0, n_feas = 0;         // (a thread evaluates far fewer than 2^32 candidates)
    u32 n_cells32 = 0;                  // splits this thread evaluated (after the early exits)
    // A search that records plans: the partition and levels of the candidate at hand go to one of two places in local
    // memory (stores that nothing waits for), the other one holds those of the thread's best candidate so far.
    __align__(16) uint8_t plan_n[2][HAP_MAX_PP], plan_r[2][HAP_MAX_PP];    // per stage: layers, level
    i64 plan_val[2][4];                 // bottleneck, T_pipe, T_sync, T_opt
    u32 plan_cur = 0;
    unsigned all_levels = 0;
    for (int q = 0; q < n_rc; ++q) all_levels |= dc.rc_masks[q];

    // ---- configurations whose first stage fits no device type at any level: nothing is feasible ----------
    // Decided before anything is staged, from the byte coefficients alone: the memory of a span is its numbers of
    // dense and MoE layers times the per-kind bytes.  Feasibility is monotone in the span, so the shortest first
    // stage the band of a depth-1 node allows decides (PP = 1: the one stage holds all N layers).
    {
        const i64 mw0 = cfp[HAP_MW], mw1 = cfp[HAP_MW + 1], ma0 = cfp[HAP_MA], ma1 = cfp[HAP_MA + 1];
        const i64 extra = cfp[HAP_MPRE] + (PP == 1 ? cfp[HAP_MPOST] : 0), mx = cfp[HAP_MX];
        const i64 mstore = pc.M < PP ? pc.M : PP;
        auto first_fits = [&](int b, i64 cap, int r) {
            const i64 nm = moe_before(dc, b), nd = (i64)b - nm;
            const i64 Wb = nd * mw0 + nm * mw1 + extra + (nm ? mx : 0);
            const i64 A = mstore * (nd * ma0 + nm * ma1);
            return Wb + (((i64)dc.xi_q[r] * A) >> 10) <= cap;
        };
        int fits = 0;
        if (PP > 1) {
            const u32 n_first = tm.node_lo[2] - tm.node_lo[1];
            for (u32 e = tid; e < n_first * (u32)R; e += nthreads) {
                const u32 nd_i = e / R; const int r = (int)(e % R);
                if (!((all_levels >> r) & 1u)) continue;
                const TrieNode nd = tm.nodes[tm.node_lo[1] + nd_i];
                if (nd.bl > nd.bh) continue;
                i64 cap = 0; bool seen = false;
                for (int h = 0; h < T; ++h)
                    if (nd.mask >> h & 1) { if (!seen || dc.cap_eff[h] < cap) cap = dc.cap_eff[h]; seen = true; }
                fits |= first_fits(nd.bl, cap, r);
            }
        } else {
            for (int e = tid; e < T * R; e += nthreads) {
                const int t = e / R, r = e % R;
                if (!((all_levels >> r) & 1u) || !((tm.tmask[1] >> t) & 1u)) continue;
                fits |= first_fits(N, dc.cap_eff[t], r);
            }
        }
        if (!__syncthreads_or(fits)) {
            // every candidate of the block is infeasible: say so and leave
            if (SEARCH) {
                if (tid == 0) {
                    out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull;
                    atomicAdd(out.counters + 0, block_candidates());
                }
            } else {
                const u64 a = c_lo > w_lo ? c_lo : w_lo, b = c_hi < w_hi ? c_hi : w_hi;
                for (u64 c = a + tid; c < b; c += nthreads) put_infeasible(c);
            }
            return;
        }
    }

    // ---- layer times of the configuration; in a pruning search whose blocks compute them, the lower bound too ----
    trie_stage_costs<VT>(dc, pc, p, c2, out.tcg, out.range_flag, sC);
    if (SEARCH && out.prune && out.tcg) {
        if (tid == 0) s_lb = 0;
        __syncthreads();
        i64 lmin = 0;
        for (int l = tid; l < N; l += nthreads) {
            i64 m = 0;
            for (int h = 0; h < T; ++h) { const i64 q = (i64)sC[((size_t)h * N + l) * 2] + (i64)sC[((size_t)h * N + l) * 2 + 1]; m = (h == 0 || q < m) ? q : m; }
            lmin += m;
        }
        lmin = warp_sum_i64(lmin);
        if (lane == 0 && lmin) atomicAdd(&s_lb, (unsigned long long)lmin);
        __syncthreads();
        if (tid == 0) {
            const i64 S = (i64)s_lb;
            const i64 lb = S + (i64)(pc.M - 1) * ((S + PP - 1) / PP);
            const u64 inc = *reinterpret_cast<volatile const u64 *>(out.incumbent);
            s_skip = (u64)lb > inc;
            if (s_skip) {
                out.partial_cost[blockIdx.x] = kInf; out.partial_index[blockIdx.x] = ~0ull;
                atomicAdd(out.counters + 2, block_candidates());
            }
        }
        __syncthreads();
        if (s_skip) return;
    }
    trie_prologue_rows<VT>(dc, tm, p, coef, coefv, sW, sA, sK, sKtab, sNodes, sParent, minfo, sP2P, szero);
    trie_prologue_time_rows<VT>(dc, tm, sC, sR);
    trie_prologue_thr(dc, pc, tm, p, coef, all_levels, sW, sA, thr, sK);

    const u32 a_thr = smem_u32(thr), a_sR = smem_u32(sR);
    const bool all_flat = tm.all_flat != 0;
    const int kind0 = layer_kind(dc, 0);

    // One cell: min over k in [klo, khi] of max(prev[k], cost(k, j)), smallest k on ties.  k runs downward over the
    // level segments given by the memory thresholds (lowest allowed level that fits); prev[k] and the time row
    // entry of k are read through two addresses that step down together, two splits per step.
    // Times are integer ns below 2^53 held as doubles: every sum, difference and comparison is exact, and the
    // subtraction and the two comparisons of a split run on the fp64 pipe instead of as int64 pairs on the ALU pipe.
    //   a_prev: address of prev[0]; a_th: address of the level-0 threshold of (stage, j); a_row: address of entry 0
    //   of the level-0 time row of the stage's types; K: stage constant
    const double dInf = 4611686018427387904.0;             // 2^62, the integer INF
    auto cell = [&](u32 a_prev, int j, int klo, int khi, u32 a_th, u32 a_row, double K, unsigned rc_mask, double &best_out, int &arg_out) {
        double best = 2305843009213693952.0;   // 2^61: every finite value is below this, an unreachable one (2^62) above
        u32 a_arg = 0;
        int seg_hi = khi;
        for (int r = 0; r < R && seg_hi >= klo; ++r, a_th += (u32)bw, a_row += (u32)n1 * 8u) {
            if (!((rc_mask >> r) & 1u)) continue;
            int lo = j - lds_u8(a_th);           // first split of this level: end layer minus the longest span that fits
            if (lo < klo) lo = klo;
            if (lo > seg_hi) continue;
            const int n = seg_hi - lo + 1;
            // integer mode: (row[j] + K) - row[k], exact in any order; fp64 mode keeps the order (row[j] - row[k]) + K
            const double Rj = lds_f64<0>(a_row + 8u * (u32)j);
            const double Cj = F64 ? Rj : Rj + K;
            const double Kadd = F64 ? K : 0.0;
            u32 pa = a_prev + 8u * (u32)seg_hi, ra = a_row + 8u * (u32)seg_hi;
            const u32 pa_lo = a_prev + 8u * (u32)lo;
            if (n & 1) {
                const double p0 = lds_f64<0>(pa), c0 = F64 ? (Cj - lds_f64<0>(ra)) + Kadd : Cj - lds_f64<0>(ra);
                const double v0 = p0 > c0 ? p0 : c0;
                if (v0 <= best) { best = v0; a_arg = pa; }
                pa -= 8; ra -= 8;
            }
            while ((int)(pa - pa_lo) > 0) {      // pa and pa - 8 are both inside the segment
                const double p0 = lds_f64<0>(pa), p1 = lds_f64<-8>(pa);
                const double c0 = F64 ? (Cj - lds_f64<0>(ra)) + Kadd : Cj - lds_f64<0>(ra);
                const double c1 = F64 ? (Cj - lds_f64<-8>(ra)) + Kadd : Cj - lds_f64<-8>(ra);
                const double v0 = p0 > c0 ? p0 : c0, v1 = p1 > c1 ? p1 : c1;
                if (v0 <= best) { best = v0; a_arg = pa; }
                if (v1 <= best) { best = v1; a_arg = pa - 8; }
                // layer times are non-negative, so the stage cost only grows as k falls within a level: once it
                // exceeds the best value no further split of this level can reach it
                if (c1 > best) { if (COUNT) pa -= 16; break; }
                pa -= 16; ra -= 16;
            }
            if (COUNT) n_cells32 += ((a_prev + 8u * (u32)seg_hi) - pa) >> 3;      // splits evaluated (pa has stepped past them)
            seg_hi = lo - 1;
        }
        best_out = a_arg ? best : dInf;
        arg_out = a_arg ? (int)((a_arg - a_prev) >> 3) : 255;
    };

    unsigned policies_without_plan = 0;                      // positions in rc_order under which no mapping was feasible
    for (int rc_pos = 0; rc_pos < n_rc; ++rc_pos) {
        const int rc_idx = dc.rc_order[rc_pos];
        const unsigned rc_mask = dc.rc_masks[rc_idx];
        bool dead = (dc.rc_sup[rc_pos] & policies_without_plan) != 0;

        // ---- rows of the tree, depth by depth ------------------------------------------------
        if (!dead) {
            // a thread's first cell record of a depth is requested before the barrier that ends the previous depth
            TrieCell nxt = make_uint4(0, 0, 0, 0);
            if (PP > 1 && (u32)tid < tm.cell_lo[2] - tm.cell_lo[1]) nxt = __ldcs(tm.cells + tm.cell_lo[1] + tid);
            for (int d = 1; d < PP; ++d) {
                const u32 ncell = tm.cell_lo[d + 1] - tm.cell_lo[d];
                const TrieCell *cells = tm.cells + tm.cell_lo[d];
                uint8_t *chd = ch + tm.cell_lo[d];
                double *cur = (d & 1) ? bufO : bufE;
                const u32 a_prevbuf = smem_u32(d == 1 ? szero : ((d & 1) ? bufE : bufO)) - 256u * 8u;
                int alive = 0;
                for (u32 e = tid; e < ncell; e += nthreads) {
                    const TrieCell rec = nxt;
                    if (e + nthreads < ncell) nxt = __ldcs(cells + e + nthreads);     // next record while this cell runs (streamed past L1)
                    const int j = rec.y & 255, klo = (rec.y >> 8) & 255, khi = (rec.y >> 16) & 255;
                    const double K = sKtab[rec.x >> 26];
                    double best; int arg;
                    (void)HAP_CHECK_OK(6, rec.z + (u32)(R - 1) * (u32)bw < (u32)thr_bytes);
                    cell(a_prevbuf + 8u * (rec.x & 0x03ffffffu), j, klo, khi, a_thr + rec.z, a_sR + 8u * rec.w, K, rc_mask, best, arg);
                    if (HAP_CHECK_OK(1, e < tm.buf_cells[d & 1])) cur[e] = best;
                    if (HAP_CHECK_OK(2, tm.cell_lo[d] + e < tm.cell_lo[PP])) chd[e] = (uint8_t)arg;
                    alive |= best < dInf;
                }
                if (d + 1 < PP && (u32)tid < tm.cell_lo[d + 2] - tm.cell_lo[d + 1]) nxt = __ldcs(tm.cells + tm.cell_lo[d + 1] + tid);
                if (!__syncthreads_or(alive)) { dead = true; break; }   // no cell of this depth is finite: nothing below is
            }
        }
        // ---- one thread per mapping: cell (PP, N), backtrace, Eq. 4 ---------------------------------
        auto stage_K = [&](int d, int mask, int link) -> VT {
            VT K = 0;
            const MaskInfo<VT> &mi = minfo[mask - 1];
            if (d == 1) K += mi.kpre;
            if (d == PP) K += mi.kpost;
            if (d > 1) { const int cls = link & 3, ha = (link >> 2) & 3, hb = (link >> 4) & 3; K += sP2P[hb][cls == HAP_CROSS ? 2 + ha : cls]; }
            return K;
        };
        int any_plan = 0;
        const u32 a_last = smem_u32(PP == 1 ? szero : (((PP - 1) & 1) ? bufO : bufE));
        for (u32 m = tid; m < tm.nmap; m += nthreads) {
            const u64 c = s_clo + (u64)m * n_rc + (u64)rc_idx;
            if (c < out.first || c >= out.first + out.count) continue;
            if (!HAP_CHECK_OK(3, c - out.first < out.count)) continue;
            double bott_d = dInf; int arg = 255;
            int mask = 0, link = 0;
            u32 node = 0;
            if (!dead) {
                const uint4 raw = __ldg(reinterpret_cast<const uint4 *>(tm.leaves + m));
                const u32 prowoff = raw.x;
                node = raw.y & 0xffff; mask = (raw.y >> 16) & 255; link = raw.y >> 24;
                const int nmin = raw.z & 255, nmax = (raw.z >> 8) & 255, pbl = (raw.z >> 16) & 255, pbh = raw.z >> 24;
                const int ldead = raw.w & 255, capt = (raw.w >> 8) & 255;
                if (!ldead) {
                    int klo = N - nmax; if (klo < pbl) klo = pbl;
                    int khi = N - nmin; if (khi > pbh) khi = pbh;
                    cell(a_last + 8u * prowoff - 8u * (u32)pbl, N, klo, khi, a_thr + trie_thr_index(tm, T, R, PP, capt, 0, N),
                         a_sR + 8u * (u32)tm.mrow_of[mask] * (u32)(R * n1), (double)stage_K(PP, mask, link), rc_mask, bott_d, arg);
                }
            }
            if (SEARCH) n_eval++;
            const VT bott = bott_d < dInf ? (VT)bott_d : vInf;
            if (!(bott < vInf)) {
                if (!SEARCH) put_infeasible(c);
                continue;
            }
            // backtrace from (PP, N) through the ancestors; per stage: level, cost, sync and optimizer terms
            VT sum = 0, mxc = 0, t_sync = 0, t_opt = 0, het = 0;
            const u64 o = c - out.first;
            int b = N, a = arg;
            double Kd = (double)stage_K(PP, mask, link);          // stage constant of the stage at hand (exact in a double)
            for (int d = PP; d >= 1; --d) {
                // the ancestor's record is fetched before this stage's arithmetic needs to wait for it
                uint4 raw = make_uint4(0, 0, 0, 0);
                u32 parent = 0;
                if (d > 1) {
                    if (!HAP_CHECK_OK(4, node < tm.node_lo[d] - tm.node_lo[d - 1])) break;
                    raw = *reinterpret_cast<const uint4 *>(sNodes + tm.node_lo[d - 1] + node);
                    parent = sParent[tm.node_lo[d - 1] + node];
                }
                if (!HAP_CHECK_OK(5, a >= 0 && a < b && b <= N && mask >= 1 && mask <= kMaxMasks)) break;
                const MaskInfo<VT> &mi = minfo[mask - 1];
                const u32 ti = all_flat ? (u32)(((d - 1) * T + mi.capt) * R) : trie_thr_index(tm, T, R, d, mi.capt, 0, b);
                if (!HAP_CHECK_OK(6, ti + (u32)(R - 1) * (u32)bw < (u32)thr_bytes)) break;
                const uint8_t *th = thr + ti;
                int r = 0;
                for (; r < R; ++r)
                    if (((rc_mask >> r) & 1u) && b - (int)th[r * bw] <= a) break;
                const int mrow = tm.mrow_of[mask];
                const double *rr = sR + ((size_t)mrow * R + r) * n1;
                const VT cst = (VT)((rr[b] - rr[a]) + Kd);
                sum += cst; mxc = cst > mxc ? cst : mxc;
                VT sy, op;
                if (dc.kind_uniform) {                               // one layer kind: the terms are a count times a coefficient
                    const VT n = (VT)(b - a);
                    sy = mi.slat + n * mi.sbw[kind0]; op = n * mi.opt[kind0];
                } else {
                    const VT n_moe = (VT)((int)sK[b] - (int)sK[a]), n_dense = (VT)(b - a) - n_moe;
                    sy = mi.slat + n_dense * mi.sbw[0] + n_moe * mi.sbw[1];
                    op = n_dense * mi.opt[0] + n_moe * mi.opt[1];
                }
                t_sync = sy > t_sync ? sy : t_sync; t_opt = op > t_opt ? op : t_opt;
                if (dc.eta_q > 0) {                                  // Pruning 3: cross-type transfer into the stage; dispatch of a mixed-type stage
                    if (d > 1 && (link & 3) == HAP_CROSS) het += sP2P[(link >> 4) & 3][2 + ((link >> 2) & 3)];
                    het += (VT)((int)sK[b] - (int)sK[a]) * mi.kxd;
                }
                if (!SEARCH) {
                    if (out.partition) out.partition[o * HAP_MAX_PP + d - 1] = (uint8_t)(b - a);
                    if (out.recompute) out.recompute[o * HAP_MAX_PP + d - 1] = (uint8_t)r;
                } else if (out.block_plan) { plan_n[plan_cur][d - 1] = (uint8_t)(b - a); plan_r[plan_cur][d - 1] = (uint8_t)r; }
                if (d > 1) {
                    b = a;
                    if (!HAP_CHECK_OK(2, b >= (int)(raw.w & 255) && raw.x + (u32)(b - (int)(raw.w & 255)) < tm.cell_lo[d] - tm.cell_lo[d - 1])) break;
                    a = ch[tm.cell_lo[d - 1] + raw.x + (u32)(b - (int)(raw.w & 255))];
                    mask = raw.z & 255; link = (raw.z >> 8) & 255;
                    node = parent;
                    // the stage constant of stage d-1 from the block's table: pre-work of a first stage by row group,
                    // transfer into a later stage by receiving type and link class (the entries the cells use)
                    const int cls = link & 3;
                    Kd = sKtab[d == 2 ? (int)tm.mrow_of[mask] : 16 + ((link >> 4) & 3) * 6 + (cls == HAP_CROSS ? 2 + ((link >> 2) & 3) : cls)];
                }
            }
            VT T_pipe = sum + (VT)(pc.M - 1) * mxc;
            VT T_iter = T_pipe + t_sync + t_opt;
            if (dc.eta_q > 0 && het * (VT)PP * (VT)1024 > (VT)dc.eta_q * sum) { T_iter = vInf; T_pipe = vInf; }   // Pruning 3
            if (SEARCH) {
                if (T_iter < vInf) { n_feas++; any_plan = 1; }
                {   // (offsets grow with the candidate index, so the smaller offset is the smaller index)
                    const u32 loc = m * (u32)n_rc + (u32)rc_idx;
                    if ((i64)T_iter < best_cost || ((i64)T_iter == best_cost && loc < best_local)) {
                        best_cost = (i64)T_iter; best_local = loc;
                        if (out.block_plan) {
                            plan_val[plan_cur][0] = (i64)bott; plan_val[plan_cur][1] = (i64)T_pipe;
                            plan_val[plan_cur][2] = (i64)t_sync; plan_val[plan_cur][3] = (i64)t_opt;
                            plan_cur ^= 1u;                  // the place just filled is kept, the other one is written next
                        }
                    }
                }
            } else {
                any_plan = 1;
                if (out.cost) reinterpret_cast<VT *>(out.cost)[o] = T_iter;
                if (out.bottleneck) reinterpret_cast<VT *>(out.bottleneck)[o] = bott;
                if (out.detail) { VT *dt = reinterpret_cast<VT *>(out.detail); dt[o * 3] = T_pipe; dt[o * 3 + 1] = t_sync; dt[o * 3 + 2] = t_opt; }
                if (!(T_iter < vInf)) {
                    if (out.partition) for (int s = 0; s < PP; ++s) out.partition[o * HAP_MAX_PP + s] = 0;
                    if (out.recompute) for (int s = 0; s < PP; ++s) out.recompute[o * HAP_MAX_PP + s] = 0;
                }
                if (out.partition) for (int s = PP; s < HAP_MAX_PP; ++s) out.partition[o * HAP_MAX_PP + s] = 0;
                if (out.recompute) for (int s = PP; s < HAP_MAX_PP; ++s) out.recompute[o * HAP_MAX_PP + s] = 0;
            }
        }
        // the barrier also keeps the next policy from overwriting rows and choices that are still being read
        const int bott_any = __syncthreads_or(any_plan);
        // a policy under which none of the block's mappings has a feasible partition settles its subsets
        if (!bott_any && s_whole && dc.eta_q <= 0) policies_without_plan |= 1u << rc_pos;
    }

    if (COUNT && out.counters) {
        const u64 n_cells = (u64)warp_sum_i64((i64)n_cells32);
        if (lane == 0 && n_cells) atomicAdd(out.counters + 4, n_cells);
    }
    if (SEARCH) {
        const u64 n_eval_w = (u64)warp_sum_i64((i64)n_eval), n_feas_w = (u64)warp_sum_i64((i64)n_feas);
        u64 best_index = best_local == ~0u ? ~0ull : s_clo + (u64)best_local;
        warp_argmin(best_cost, best_index);
        if (lane == 0) {
            wcost[wib] = best_cost; widx[wib] = best_index;
            if (n_eval_w) atomicAdd(out.counters + 0, n_eval_w);
            if (n_feas_w) atomicAdd(out.counters + 1, n_feas_w);
        }
        __syncthreads();
        if (tid == 0) {
            i64 bc = wcost[0]; u64 bi = widx[0];
            for (int q = 1; q < nwarps; ++q)
                if (wcost[q] < bc || (wcost[q] == bc && widx[q] < bi)) { bc = wcost[q]; bi = widx[q]; }
            out.partial_cost[blockIdx.x] = bc;
            out.partial_index[blockIdx.x] = bi;
            if (out.prune && bc < kInf) atomicMin(out.incumbent, (u64)bc);
            wcost[0] = bc; widx[0] = bi;
        }
        if (out.block_plan) {
            // the thread that evaluated the block's best candidate writes its plan to the block's slot
            __syncthreads();
            if (wcost[0] < kInf && best_local != ~0u && s_clo + (u64)best_local == widx[0]) {
                PlanSlot *ps = out.block_plan + blockIdx.x;
                const u32 keep = plan_cur ^ 1u;
                ps->bott = plan_val[keep][0]; ps->T_pipe = plan_val[keep][1]; ps->T_sync = plan_val[keep][2]; ps->T_opt = plan_val[keep][3];
                ps->PP = PP;                                  // (entries of later stages are whatever the thread's memory held)
                const uint4 *sn = reinterpret_cast<const uint4 *>(plan_n[keep]), *sr = reinterpret_cast<const uint4 *>(plan_r[keep]);
                uint4 *dn = reinterpret_cast<uint4 *>(ps->n), *dr = reinterpret_cast<uint4 *>(ps->r);
                dn[0] = sn[0]; dr[0] = sr[0];
                if (PP > 16) { dn[1] = sn[1]; dr[1] = sr[1]; }
            }
        }
    }
}

}  // namespace hap

// Host side of libhap: descriptor validation and copies, enumeration of the 6-D space,
// work partitioning, kernel launches.  Every step of the hot path runs in the kernels of
// hap_device.cuh; nothing here evaluates a cost.
#include "hap_device.cuh"
#include "hap_trie.cuh"

#include <algorithm>
#include <cstdarg>
#include <cstdio>
#include <cmath>
#include <cstring>
#include <array>
#include <map>
#include <memory>
#include <mutex>
#include <new>
#include <string>
#include <unordered_map>
#include <vector>
#if defined(__SSE2__)
#include <emmintrin.h>
#endif

using namespace hap;

// read-only view of a vector that someone else keeps alive
template <typename E> struct View {
    const E *ptr = nullptr;
    size_t n = 0;
    size_t size() const { return n; }
    bool empty() const { return n == 0; }
    const E *data() const { return ptr; }
    const E &operator[](size_t i) const { return ptr[i]; }
    const E *begin() const { return ptr; }
    const E *end() const { return ptr + n; }
};

struct hap_problem {
    int device = 0;
    // host copies
    hap_model model{};
    std::vector<uint8_t> kind;
    int T = 0;
    std::vector<int64_t> P, C, cap_eff;
    std::vector<int32_t> node_size, node_type, tp_list, cp_list, mb_list, ep_list, pp_list, tpe_list, xi_q, tau_q;
    std::vector<double> bw_intra, node_bw_inter, eta, croute, alpha, rho, act_coef, copt;
    std::vector<uint32_t> rc_masks;
    hap_profile prof{};
    hap_search_opts opts{};
    int64_t m[HAP_MAX_TYPES] = {0, 0, 0, 0};
    int64_t W = 0;
    // enumeration: the configuration table and the work items belong to the per-process enumeration result that
    // `enum_ref` keeps alive (problems with the same lists share one)
    bool enumerated = false;
    View<hap_pconf> pconfs;
    uint64_t n_cand = 0;
    View<WorkItem> items;                  // grouped by PP class, heaviest class first
    std::shared_ptr<const void> enum_ref;
    std::shared_ptr<const void> tree_image;      // the page-locked image the trees were uploaded from (kept until the copy is known to be done)
    // prefix tree of a class's mappings (trie_dp_kernel); ok = false: the class runs in pipeline_dp_kernel only
    struct TriePartDev { TrieNode *d_nodes; TrieLeaf *d_leaves; TrieCell *d_cells; u32 *d_first_leaf, *d_gnode; uint8_t *d_depth;
                         u32 n_nodes, n_cells, nmap, m_lo; uint8_t mrow_of[16]; };
    struct Trie { bool ok = false; TrieMeta *d_metas = nullptr; u32 *d_plist = nullptr;       // both inside d_trie_arena
                  std::vector<TriePartDev> parts; unsigned n_conf = 0; int threads = 0; size_t smem = 0; };
    struct PpClass { int PP; int warps; size_t smem; size_t item_lo, item_hi; u64 map_base; bool has_tab; bool multiset; unsigned masks_used; cudaStream_t stream; cudaEvent_t done; Trie trie;
                     mutable bool tab_valid = false;        // the device table of decoded mappings of this class has been filled
                     size_t pslot_lo = 0, pslot_n = 0; };   // the class's slots in the per-block partial minima of a search
    std::vector<PpClass> classes;
    uint8_t *d_maptab = nullptr;           // decoded mappings of every class that is small enough
    unsigned char *d_arena = nullptr;      // everything hap_enumerate sizes, in one allocation (the d_* pointers below point into it)
    unsigned char *d_trie_arena = nullptr; // the prefix trees of all classes
    // device
    DevConst dc{};
    double *d_tables = nullptr;            // all six tables in one allocation
    hap_pconf *d_pconf = nullptr;
    WorkItem *d_items = nullptr;
    i64 *d_c2 = nullptr, *d_coef = nullptr;
    double *d_c2f = nullptr, *d_coeff = nullptr;   // fp64-mode layer costs and coefficients (allocated on first use)
    i64 *d_fcost = nullptr;                 // fp64-mode search: per-candidate costs (bit patterns), allocated on first use
    u64 *d_range = nullptr;                 // sticky flag: a cost left the supported value range
    // joint device-state recurrence (built on first use)
    struct JointHost { JointClass jc; std::vector<unsigned> ids; unsigned *d_ids = nullptr; int *d_arrays = nullptr; size_t smem = 0; };
    std::vector<JointHost> joint;
    i64 *d_joint_scratch = nullptr;
    int joint_grid = 0;
    bool joint_ready = false;
    i64 *d_lb = nullptr;                    // scratch: per-configuration lower bound on the summed stage time
    PlanSlot *d_plans = nullptr;            // per partial-minimum slot the plan of the block's best candidate (searches over the prefix trees; first use)
    i64 *d_cand_lb = nullptr;               // scratch of the refinement searches: per-candidate bottleneck, then lower bound (first use)
    TypeConst *d_tc = nullptr;              // scratch: per (configuration, type) constants of the layer-cost kernels
    i64 *d_pcost = nullptr;                // per-block partial minima
    u64 *d_pindex = nullptr;
    u64 *d_counters = nullptr;             // [0] evaluated [1] feasible [2] pruned [3] incumbent
    i64 *d_best = nullptr;                 // (cost, index) of the search
    void *d_single = nullptr;              // outputs of the one-candidate re-evaluation
    size_t n_partial = 0;                  // allocated slots of the partial minima
    size_t n_pslots = 0;                   // slots a search pass writes and reduces (sum of the classes' pslot_n)
    bool timed = false;
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};
    cudaEvent_t ev_upload = nullptr;       // the last host-to-device upload of this problem (tables, configuration table, trees)
    bool upload_pending = false;           // that upload has not been waited for yet
    cudaEvent_t ev_fork = nullptr;          // classes run on their own streams between this event and their `done` events
    cudaEvent_t ev_pre = nullptr;           // start of a pass: the candidate decode of the classes waits for this one only
    cudaEvent_t ev_dec = nullptr;           // the merged candidate decode of a pass has finished
    DecodeJobs decode_jobs{};               // classes that walk a prefix tree: one merged decode launch per pass
    GatherJob *d_gather_jobs = nullptr;     // inside d_trie_arena: one entry per part of every tree
    int n_gather_jobs = 0;
    unsigned gather_blocks = 0;
    bool decoded_all = false;               // this pass's merged decode is already queued
    std::string err;
};

// device-side landing area of the one-candidate re-evaluation that fills the plan
struct SingleOut {
    i64 cost, bott, detail[3];
    uint8_t part[HAP_MAX_PP], rec[HAP_MAX_PP];
    hap_candidate cand;
};

// The side streams the PP classes run on are shared by all problems of a device and live until the process ends:
// creating half a dozen streams costs more than a whole search.  Index = position of the class in the problem,
// classes ordered from the deepest pipeline down.  A block of a deep class is a long chain of short steps (one
// barrier-separated depth of its tree per stage and policy) that leaves most issue slots idle, a block of the class
// with the most mappings keeps them busy but fills an SM's registers: the deep classes' blocks should be resident
// first and the busy class should fill in behind them, so the streams get priorities in class order: the phase is
// shorter and takes the same time in every pass.
static cudaStream_t pooled_stream(int device, size_t index)
{
    static std::mutex mu;
    static cudaStream_t pool[64][HAP_MAX_PP + 1];
    std::lock_guard<std::mutex> lock(mu);
    cudaStream_t &s = pool[device & 63][index % (HAP_MAX_PP + 1)];
    if (!s) {
        int least = 0, greatest = 0;                    // numerically: greatest priority <= least priority
        if (cudaDeviceGetStreamPriorityRange(&least, &greatest) != cudaSuccess) { least = greatest = 0; cudaGetLastError(); }
        const int pr = std::min(least, greatest + (int)(index % (HAP_MAX_PP + 1)));
        if (cudaStreamCreateWithPriority(&s, cudaStreamNonBlocking, pr) != cudaSuccess) s = nullptr;
    }
    return s;
}

// Uploads (profiled tables, configuration table, prefix trees) go through page-locked staging buffers and an
// upload stream of their own, asynchronously: the host builds the next thing while the copy runs, and the first call
// that uses the data waits for the upload's event.  The staging buffers are kept per process (a page-locked
// allocation costs more than a search); a buffer is reused once the copy that last read it has completed.
namespace {
struct PinnedBuf { void *ptr = nullptr; size_t cap = 0; cudaEvent_t done = nullptr; int device = -1; };
struct UploadState {
    std::mutex mu;
    std::vector<PinnedBuf> bufs;
    cudaStream_t stream[64] = {};
};
UploadState &upload_state() { static UploadState *u = new UploadState(); return *u; }      // never destroyed
constexpr size_t kPinnedBufs = 8;
}  // namespace

static cudaStream_t upload_stream(int device)
{
    UploadState &u = upload_state();
    std::lock_guard<std::mutex> lock(u.mu);
    cudaStream_t &s = u.stream[device & 63];
    if (!s && cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess) s = nullptr;
    return s;
}

// a page-locked buffer of at least `bytes` whose previous copy (if any) has completed; nullptr: use pageable memory
static PinnedBuf *pinned_get(int device, size_t bytes)
{
    UploadState &u = upload_state();
    std::lock_guard<std::mutex> lock(u.mu);
    for (auto &b : u.bufs)
        if (b.device == device && b.cap >= bytes && cudaEventQuery(b.done) == cudaSuccess) return &b;
    cudaGetLastError();                                  // cudaErrorNotReady of a busy buffer is not an error
    if (u.bufs.size() >= kPinnedBufs) {                  // reuse the oldest buffer of the device: wait for it, regrow it
        for (auto &b : u.bufs)
            if (b.device == device) {
                cudaEventSynchronize(b.done);
                if (b.cap >= bytes) return &b;
                cudaFreeHost(b.ptr); b.ptr = nullptr; b.cap = 0;
                if (cudaHostAlloc(&b.ptr, bytes, cudaHostAllocDefault) != cudaSuccess) { cudaGetLastError(); b.ptr = nullptr; return nullptr; }
                b.cap = bytes;
                return &b;
            }
        return nullptr;
    }
    u.bufs.reserve(kPinnedBufs);                          // pointers into the vector stay valid
    PinnedBuf b;
    b.device = device;
    b.cap = std::max<size_t>(bytes, 1 << 20);
    if (cudaHostAlloc(&b.ptr, b.cap, cudaHostAllocDefault) != cudaSuccess) { cudaGetLastError(); return nullptr; }
    if (cudaEventCreateWithFlags(&b.done, cudaEventDisableTiming) != cudaSuccess) { cudaFreeHost(b.ptr); cudaGetLastError(); return nullptr; }
    u.bufs.push_back(b);
    return &u.bufs.back();
}

// host -> device copy of `bytes` that `fill` writes into a staging buffer; asynchronous when a page-locked buffer
// and the upload stream are available (the problem's upload event then marks its completion), synchronous otherwise
template <class Fill>
static cudaError_t upload(hap_problem *p, void *dst, size_t bytes, Fill fill)
{
    cudaStream_t us = upload_stream(p->device);
    PinnedBuf *pb = us ? pinned_get(p->device, bytes) : nullptr;
    if (!pb) {
        std::vector<unsigned char> stage(bytes, 0);
        if (!fill(stage.data())) return cudaErrorInvalidValue;
        return cudaMemcpy(dst, stage.data(), bytes, cudaMemcpyHostToDevice);
    }
    if (!fill(static_cast<unsigned char *>(pb->ptr))) return cudaErrorInvalidValue;
    cudaError_t e = cudaMemcpyAsync(dst, pb->ptr, bytes, cudaMemcpyHostToDevice, us);
    if (e != cudaSuccess) return e;
    if ((e = cudaEventRecord(pb->done, us)) != cudaSuccess) return e;
    if (!p->ev_upload && (e = cudaEventCreateWithFlags(&p->ev_upload, cudaEventDisableTiming)) != cudaSuccess) return e;
    if ((e = cudaEventRecord(p->ev_upload, us)) != cudaSuccess) return e;
    p->upload_pending = true;
    return cudaSuccess;
}

// A host image in page-locked memory that uploads read directly, without the pass through a staging buffer: what is
// derived from the lists and the cluster alone (configuration table, prefix trees) is laid out once per process.
struct PinnedImage {
    void *ptr = nullptr;
    size_t bytes = 0;
    PinnedImage() = default;
    PinnedImage(const PinnedImage &) = delete;
    PinnedImage &operator=(const PinnedImage &) = delete;
    ~PinnedImage() { if (ptr) { cudaFreeHost(ptr); cudaGetLastError(); } }
};

static std::shared_ptr<PinnedImage> pinned_image(size_t bytes)
{
    auto im = std::make_shared<PinnedImage>();
    if (cudaHostAlloc(&im->ptr, std::max<size_t>(bytes, 1), cudaHostAllocPortable) != cudaSuccess) { cudaGetLastError(); im->ptr = nullptr; return nullptr; }
    im->bytes = bytes;
    return im;
}

// host -> device copy straight from such an image (the problem holds a reference to it until it is destroyed, which
// waits for the copy)
static cudaError_t upload_image(hap_problem *p, void *dst, const PinnedImage &im, size_t bytes)
{
    cudaStream_t us = upload_stream(p->device);
    if (!us) return cudaMemcpy(dst, im.ptr, bytes, cudaMemcpyHostToDevice);
    cudaError_t e = cudaMemcpyAsync(dst, im.ptr, bytes, cudaMemcpyHostToDevice, us);
    if (e != cudaSuccess) return e;
    if (!p->ev_upload && (e = cudaEventCreateWithFlags(&p->ev_upload, cudaEventDisableTiming)) != cudaSuccess) return e;
    if ((e = cudaEventRecord(p->ev_upload, us)) != cudaSuccess) return e;
    p->upload_pending = true;
    return cudaSuccess;
}

// the first use of uploaded data waits for the upload (on the host: by then the copy has long finished)
static cudaError_t uploads_done(hap_problem *p)
{
    if (!p->upload_pending) return cudaSuccess;
    p->upload_pending = false;
    return cudaEventSynchronize(p->ev_upload);
}

// Device memory of destroyed problems is kept for the next problem of the process: allocating and freeing the
// three arenas of a problem costs about as much as the search itself.  A freed block serves a later request
// of its device that it fits with at most a quarter (plus 1 MiB) to spare.  At most kCacheBlocks blocks and kCacheBytes
// bytes are held; hap_release_cached_memory() returns everything to the driver.
namespace {
struct CachedBlock { int device; size_t bytes; void *ptr; };
struct MemCache {
    std::mutex mu;
    std::vector<CachedBlock> idle;
    std::unordered_map<void *, CachedBlock> live;
    size_t idle_bytes = 0;
};
constexpr size_t kCacheBlocks = 24;
constexpr size_t kCacheBytes = 4ull << 30;
MemCache &mem_cache() { static MemCache *c = new MemCache(); return *c; }     // never destroyed: outlives static teardown
}  // namespace

static cudaError_t cached_malloc(int device, void **out, size_t bytes)
{
    MemCache &mc = mem_cache();
    bytes = (std::max<size_t>(bytes, 1) + 0xffff) & ~(size_t)0xffff;
    std::lock_guard<std::mutex> lock(mc.mu);
    size_t best = mc.idle.size();
    for (size_t i = 0; i < mc.idle.size(); ++i) {
        const CachedBlock &b = mc.idle[i];
        if (b.device != device || b.bytes < bytes || b.bytes > bytes + bytes / 4 + (1u << 20)) continue;
        if (best == mc.idle.size() || b.bytes < mc.idle[best].bytes) best = i;
    }
    if (best != mc.idle.size()) {
        const CachedBlock b = mc.idle[best];
        mc.idle.erase(mc.idle.begin() + (long)best);
        mc.idle_bytes -= b.bytes;
        mc.live[b.ptr] = b;
        *out = b.ptr;
        return cudaSuccess;
    }
    void *ptr = nullptr;
    cudaError_t e = cudaMalloc(&ptr, bytes);
    if (e == cudaErrorMemoryAllocation) {           // give the idle blocks of this device back and try once more
        cudaGetLastError();
        for (size_t i = mc.idle.size(); i-- > 0;)
            if (mc.idle[i].device == device) { cudaFree(mc.idle[i].ptr); mc.idle_bytes -= mc.idle[i].bytes; mc.idle.erase(mc.idle.begin() + (long)i); }
        e = cudaMalloc(&ptr, bytes);
    }
    if (e != cudaSuccess) { *out = nullptr; return e; }
    mc.live[ptr] = CachedBlock{device, bytes, ptr};
    *out = ptr;
    return cudaSuccess;
}

// The caller has made sure that no work that touches the block is still in flight.
static void cached_free(void *ptr)
{
    if (!ptr) return;
    MemCache &mc = mem_cache();
    std::lock_guard<std::mutex> lock(mc.mu);
    auto it = mc.live.find(ptr);
    if (it == mc.live.end()) { cudaFree(ptr); return; }
    const CachedBlock b = it->second;
    mc.live.erase(it);
    if (mc.idle.size() >= kCacheBlocks || mc.idle_bytes + b.bytes > kCacheBytes) { cudaFree(ptr); return; }
    mc.idle.push_back(b);
    mc.idle_bytes += b.bytes;
}

extern "C" hap_status hap_release_cached_memory(void)
{
    MemCache &mc = mem_cache();
    std::lock_guard<std::mutex> lock(mc.mu);
    int prev = 0;
    const bool have_prev = cudaGetDevice(&prev) == cudaSuccess;
    hap_status st = HAP_OK;
    for (const CachedBlock &b : mc.idle)
        if (cudaSetDevice(b.device) != cudaSuccess || cudaFree(b.ptr) != cudaSuccess) st = HAP_E_CUDA;
    mc.idle.clear();
    mc.idle_bytes = 0;
    if (have_prev) cudaSetDevice(prev);
    if (st != HAP_OK) cudaGetLastError();
    return st;
}

static hap_status fail(hap_problem *p, hap_status s, const char *fmt, ...)
{
    if (p) {
        char buf[512];
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(buf, sizeof(buf), fmt, ap);
        va_end(ap);
        p->err = buf;
    }
    return s;
}

static hap_status argmin_launch(hap_problem *p, const hap::i64 *dev_cost, uint64_t count, hap::i64 *dev_out, cudaStream_t st, hap::i64 init);

#define CUDA_TRY(p, call)                                                                          \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess)                                                                     \
            return fail(p, e_ == cudaErrorMemoryAllocation ? HAP_E_NOMEM : HAP_E_CUDA, "%s: %s", #call, \
                        cudaGetErrorString(e_));                                                   \
    } while (0)

extern "C" const char *hap_status_str(hap_status s)
{
    switch (s) {
    case HAP_OK: return "HAP_OK";
    case HAP_E_INVALID: return "HAP_E_INVALID";
    case HAP_E_NOMEM: return "HAP_E_NOMEM";
    case HAP_E_CUDA: return "HAP_E_CUDA";
    case HAP_E_RANGE: return "HAP_E_RANGE";
    case HAP_E_STATE: return "HAP_E_STATE";
    case HAP_E_INFEASIBLE: return "HAP_E_INFEASIBLE";
    }
    return "HAP_E_?";
}

extern "C" const char *hap_last_error(const hap_problem *p) { return p ? p->err.c_str() : "null problem"; }

static void release_device(hap_problem *p)
{
    // nothing of this problem may still be running when its memory goes back to the cache
    if (p->upload_pending) { cudaEventSynchronize(p->ev_upload); p->upload_pending = false; }
    if (p->d_tables || p->d_arena) cudaDeviceSynchronize();
    cached_free(p->d_tables); cached_free(p->d_arena); cached_free(p->d_trie_arena);
    cached_free(p->d_joint_scratch);
    for (auto &j : p->joint) { cached_free(j.d_ids); cached_free(j.d_arrays); }
    cached_free(p->d_c2f); cached_free(p->d_coeff); cached_free(p->d_fcost); cached_free(p->d_cand_lb); cached_free(p->d_plans);
    for (auto &e : p->ev) if (e) cudaEventDestroy(e);
    if (p->ev_fork) cudaEventDestroy(p->ev_fork);
    if (p->ev_pre) cudaEventDestroy(p->ev_pre);
    if (p->ev_dec) cudaEventDestroy(p->ev_dec);
    if (p->ev_upload) cudaEventDestroy(p->ev_upload);
    for (auto &cl : p->classes) { if (cl.done) cudaEventDestroy(cl.done); }      // the class streams belong to the pool
}

extern "C" void hap_problem_destroy(hap_problem *p)
{
    if (!p) return;
    cudaSetDevice(p->device);
    release_device(p);
    delete p;
}

template <class T>
static bool copy_list(std::vector<T> &dst, const T *src, int n)
{
    if (n < 0 || (n > 0 && !src)) return false;
    dst.assign(src, src + n);
    return true;
}

static bool finite_nonneg(const std::vector<double> &v)
{
    for (double x : v) if (!(x >= 0.0) || x > 1e300) return false;
    return true;
}

extern "C" hap_status hap_problem_create(const hap_model *mo, const hap_cluster *cl, const hap_profile *pf,
                                         const hap_search_opts *so, hap_problem **out)
{
    if (!out) return HAP_E_INVALID;
    *out = nullptr;
    if (!mo || !cl || !pf || !so) return HAP_E_INVALID;
    hap_problem *p = new (std::nothrow) hap_problem();
    if (!p) return HAP_E_NOMEM;
    // the problem is handed back even on failure paths below only through *out on success
    struct Guard { hap_problem *p; bool keep = false; ~Guard() { if (!keep) { release_device(p); delete p; } } } guard{p};

    // ---- validate and copy ------------------------------------------------------------------
    const int N = mo->N, T = cl->n_types;
    if (N < 1 || N > HAP_MAX_LAYERS || !mo->kind) return HAP_E_INVALID;
    if (T < 1 || T > HAP_MAX_TYPES || cl->n_nodes < 1) return HAP_E_INVALID;
    if ((int64_t)mo->GB * mo->N > (1ll << 22)) return HAP_E_RANGE;     // keeps M * sum of layer times below 2^62
    if (mo->S < 1 || mo->H < 1 || mo->E < 1 || mo->k < 1 || mo->nq < 1 || mo->nkv < 1 || mo->GB < 1 || mo->V < 0 ||
        mo->n_shared < 0 || mo->F_dense < 0 || mo->F_exp < 0 || !(mo->beta > 0.0) || mo->nq % mo->nkv != 0)
        return HAP_E_INVALID;
    if (pf->ntp < 1 || pf->ncp < 1 || pf->nmb < 1 || pf->nep < 1 || pf->ntp > HAP_MAX_LIST || pf->ncp > HAP_MAX_LIST ||
        pf->nmb > HAP_MAX_LIST || pf->nep > HAP_MAX_LIST || pf->R < 1 || pf->R > HAP_MAX_RC)
        return HAP_E_INVALID;
    if (so->npp < 1 || so->npp > HAP_MAX_LIST || so->ntpe < 1 || so->ntpe > HAP_MAX_LIST || so->n_rc < 1 ||
        so->n_rc > HAP_MAX_RC_MASKS || so->map_cap < 1 || so->map_cap > (1ull << 56) || so->delta_q >= 1024)
        return HAP_E_INVALID;
    p->model = *mo;
    p->kind.assign(mo->kind, mo->kind + N);
    p->model.kind = nullptr;
    for (uint8_t kd : p->kind) if (kd > 1) return HAP_E_INVALID;
    p->T = T;
    bool ok = copy_list(p->P, cl->P, T) && copy_list(p->C, cl->C, T) && copy_list(p->node_size, cl->node_size, T) &&
              copy_list(p->bw_intra, cl->bw_intra, T) && copy_list(p->node_type, cl->node_type, cl->n_nodes) &&
              copy_list(p->node_bw_inter, cl->node_bw_inter, cl->n_nodes) &&
              copy_list(p->tp_list, pf->tp_list, pf->ntp) && copy_list(p->cp_list, pf->cp_list, pf->ncp) &&
              copy_list(p->mb_list, pf->mb_list, pf->nmb) && copy_list(p->ep_list, pf->ep_list, pf->nep) &&
              copy_list(p->eta, pf->eta, T) && copy_list(p->croute, pf->croute, T) && copy_list(p->alpha, pf->alpha, 3) &&
              copy_list(p->rho, pf->rho, pf->nep) && copy_list(p->act_coef, pf->act_coef, 2) &&
              copy_list(p->copt, pf->copt, T) && copy_list(p->cap_eff, pf->cap_eff, T) &&
              copy_list(p->xi_q, pf->xi_q, pf->R) && copy_list(p->tau_q, pf->tau_q, pf->R) &&
              copy_list(p->pp_list, so->pp_list, so->npp) && copy_list(p->tpe_list, so->tpe_list, so->ntpe) &&
              copy_list(p->rc_masks, so->rc_masks, so->n_rc);
    if (!ok || !pf->tdf || !pf->tdb || !pf->tff || !pf->tfb || !pf->tpre || !pf->tpost) return HAP_E_INVALID;
    p->prof = *pf;
    p->opts = *so;
    for (int h = 0; h < T; ++h) {
        if (p->P[h] < 1 || p->P[h] > (1ll << 40) || p->node_size[h] < 1 || !(p->bw_intra[h] > 0.0) || p->cap_eff[h] < 0 ||
            !(p->eta[h] > 0.0))
            return HAP_E_INVALID;
    }
    double bw_inter[HAP_MAX_TYPES];
    bool has[HAP_MAX_TYPES] = {false, false, false, false};
    for (int n = 0; n < cl->n_nodes; ++n) {
        const int t = p->node_type[n];
        if (t < 0 || t >= T || !(p->node_bw_inter[n] > 0.0)) return HAP_E_INVALID;
        p->m[t] += p->node_size[t];
        bw_inter[t] = has[t] ? std::min(bw_inter[t], p->node_bw_inter[n]) : p->node_bw_inter[n];
        has[t] = true;
    }
    for (int h = 0; h < T; ++h) { if (!has[h]) return HAP_E_INVALID; p->W += p->m[h]; }
    auto positive = [](const std::vector<int32_t> &v) { for (int x : v) if (x < 1) return false; return true; };
    for (size_t i = 0; i < p->pp_list.size(); ++i)                   // a repeated PP would enumerate its configurations twice
        for (size_t j = 0; j < i; ++j) if (p->pp_list[i] == p->pp_list[j]) return HAP_E_INVALID;
    if (!positive(p->tp_list) || !positive(p->cp_list) || !positive(p->mb_list) || !positive(p->ep_list) ||
        !positive(p->pp_list) || !positive(p->tpe_list))
        return HAP_E_INVALID;
    for (int r = 0; r < pf->R; ++r) if (p->xi_q[r] < 0 || p->tau_q[r] < 0 || p->xi_q[r] > (1 << 20) || p->tau_q[r] > (1 << 20)) return HAP_E_INVALID;
    for (uint32_t mk : p->rc_masks) if (mk == 0 || mk >= (1u << pf->R)) return HAP_E_INVALID;
    if (!finite_nonneg(p->croute) || !finite_nonneg(p->alpha) || !finite_nonneg(p->act_coef) || !finite_nonneg(p->copt) ||
        !(pf->kappa >= 0.0) || !(pf->chi > 0.0) || !(pf->gamma >= 0.0) || !(pf->ovl_tp >= 0.0) || !(pf->ovl_cp >= 0.0) ||
        !(pf->ovl_dp >= 0.0) || !(pf->capf >= 0.0))
        return HAP_E_INVALID;
    for (double r : p->rho) if (!(r >= 1.0)) return HAP_E_INVALID;
    if (pf->n_fsize < 0 || pf->n_fsize > HAP_MAX_LIST || (pf->n_fsize > 0 && (!pf->fsize || !pf->feff))) return HAP_E_INVALID;
    for (int i = 0; i < pf->n_fsize; ++i) {
        if (!(pf->fsize[i] > 0.0) || !std::isfinite(pf->fsize[i]) || (i > 0 && !(pf->fsize[i] > pf->fsize[i - 1]))) return HAP_E_INVALID;
        for (int c = 0; c < 3; ++c) { const double e = pf->feff[c * pf->n_fsize + i]; if (!(e > 0.0 && e <= 1.0)) return HAP_E_INVALID; }
    }

    const size_t n4 = (size_t)T * pf->ntp * pf->ncp * pf->nmb, n5 = n4 * N;
    // device layout: the four per-layer tables interleaved entry by entry (one 32-byte record per (type, row, layer):
    // the layer-cost kernel reads a record with two 16-byte loads), then tpre, then tpost
    const size_t n_tab = 4 * n5 + 2 * n4;
    auto fill_tables = [&](unsigned char *dst) -> bool {
        double *__restrict__ tables = reinterpret_cast<double *>(dst);
        const double *__restrict__ A = pf->tdf, *__restrict__ B = pf->tdb, *__restrict__ F = pf->tff, *__restrict__ G = pf->tfb;
        bool ok = true;
        size_t i = 0;
        // t_dense includes its FFN; every entry finite, non-negative, < 2^50 ns (NaN fails every comparison)
#if defined(__SSE2__)
        {   // two entries per step: the records are the 2 x 2 transposes of the four streams
            const __m128d zero = _mm_setzero_pd(), big = _mm_set1_pd(1e15);
            __m128d okv = _mm_castsi128_pd(_mm_set1_epi32(-1));
            for (; i + 2 <= n5; i += 2) {
                const __m128d a = _mm_loadu_pd(A + i), b = _mm_loadu_pd(B + i), c = _mm_loadu_pd(F + i), d = _mm_loadu_pd(G + i);
                double *rec = tables + 4 * i;
                _mm_storeu_pd(rec, _mm_unpacklo_pd(a, b)); _mm_storeu_pd(rec + 2, _mm_unpacklo_pd(c, d));
                _mm_storeu_pd(rec + 4, _mm_unpackhi_pd(a, b)); _mm_storeu_pd(rec + 6, _mm_unpackhi_pd(c, d));
                __m128d v = _mm_and_pd(_mm_cmpge_pd(a, c), _mm_cmpge_pd(b, d));
                v = _mm_and_pd(v, _mm_and_pd(_mm_cmpge_pd(c, zero), _mm_cmpge_pd(d, zero)));
                v = _mm_and_pd(v, _mm_and_pd(_mm_cmple_pd(a, big), _mm_cmple_pd(b, big)));
                okv = _mm_and_pd(okv, v);
            }
            ok = _mm_movemask_pd(okv) == 3;
        }
#endif
        for (; i < n5; ++i) {
            const double a = A[i], b = B[i], c = F[i], d = G[i];
            double *rec = tables + 4 * i;
            rec[0] = a; rec[1] = b; rec[2] = c; rec[3] = d;
            ok &= (a >= c) & (b >= d) & (c >= 0.0) & (d >= 0.0) & (a <= 1e15) & (b <= 1e15);
        }
        for (size_t i = 0; i < n4; ++i) {
            const double a = pf->tpre[i], b = pf->tpost[i];
            tables[4 * n5 + i] = a; tables[4 * n5 + n4 + i] = b;
            ok &= (a >= 0.0) & (b >= 0.0) & (a <= 1e15) & (b <= 1e15);
        }
        return ok;
    };

    // ---- device ------------------------------------------------------------------------------
    if (cudaGetDevice(&p->device) != cudaSuccess) return HAP_E_CUDA;
    if (cached_malloc(p->device, (void **)&p->d_tables, n_tab * sizeof(double)) != cudaSuccess) return HAP_E_NOMEM;
    {
        const cudaError_t e = upload(p, p->d_tables, n_tab * sizeof(double), fill_tables);
        if (e == cudaErrorInvalidValue) { cudaGetLastError(); return HAP_E_INVALID; }
        if (e != cudaSuccess) return HAP_E_CUDA;
    }
    for (auto &e : p->ev) if (cudaEventCreate(&e) != cudaSuccess) return HAP_E_CUDA;

    DevConst &dc = p->dc;
    std::memset(&dc, 0, sizeof(dc));
    dc.N = N; dc.T = T; dc.R = pf->R; dc.n_rc = so->n_rc; dc.ntp = pf->ntp; dc.ncp = pf->ncp; dc.nmb = pf->nmb; dc.nep = pf->nep;
    dc.S = mo->S; dc.H = mo->H; dc.E = mo->E; dc.k = mo->k; dc.n_shared = mo->n_shared; dc.F_dense = mo->F_dense;
    dc.F_exp = mo->F_exp; dc.nq = mo->nq; dc.nkv = mo->nkv; dc.V = mo->V; dc.GB = mo->GB; dc.delta_q = so->delta_q; dc.eta_q = so->eta_q; dc.uniform = (so->flags & HAP_OPT_UNIFORM) != 0;
    dc.het_dispatch = (so->flags & HAP_OPT_HETERO_DISPATCH) != 0;
    dc.beta = mo->beta; dc.kappa = pf->kappa; dc.chi = pf->chi; dc.gamma = pf->gamma; dc.ovl_tp = pf->ovl_tp;
    dc.ovl_cp = pf->ovl_cp; dc.ovl_dp = pf->ovl_dp; dc.capf = pf->capf;
    for (int i = 0; i < 3; ++i) dc.alpha[i] = p->alpha[i];
    for (int h = 0; h < T; ++h) {
        dc.eta[h] = p->eta[h]; dc.croute[h] = p->croute[h]; dc.copt[h] = p->copt[h]; dc.bw_intra[h] = p->bw_intra[h];
        dc.bw_inter[h] = bw_inter[h]; dc.P[h] = p->P[h]; dc.cap_eff[h] = p->cap_eff[h]; dc.m[h] = p->m[h];
        dc.node_size[h] = p->node_size[h];
    }
    dc.act_coef[0] = p->act_coef[0]; dc.act_coef[1] = p->act_coef[1];
    for (int i = 0; i < pf->nep; ++i) dc.rho[i] = p->rho[i];
    for (int i = 0; i < so->n_rc; ++i) dc.rc_masks[i] = p->rc_masks[i];
    {   // evaluation order of the policies: more allowed levels first (stable), and who contains whom
        std::vector<int> order(so->n_rc);
        for (int i = 0; i < so->n_rc; ++i) order[i] = i;
        std::stable_sort(order.begin(), order.end(), [&](int a, int b) {
            return __builtin_popcount(p->rc_masks[a]) > __builtin_popcount(p->rc_masks[b]);
        });
        for (int j = 0; j < so->n_rc; ++j) {
            dc.rc_order[j] = order[j];
            dc.rc_sup[j] = 0;
            for (int q = 0; q < j; ++q)
                if ((p->rc_masks[order[q]] & p->rc_masks[order[j]]) == p->rc_masks[order[j]]) dc.rc_sup[j] |= 1u << q;
        }
    }
    dc.n_fsize = pf->n_fsize;
    for (int i = 0; i < pf->n_fsize; ++i) {
        dc.fsize[i] = pf->fsize[i];
        for (int c = 0; c < 3; ++c) dc.feff[c][i] = pf->feff[c * pf->n_fsize + i];
    }
    dc.tau_linear = 1;
    for (int r = 0; r < pf->R; ++r) { dc.xi_q[r] = p->xi_q[r]; dc.tau_q[r] = p->tau_q[r]; if (p->tau_q[r] % 1024) dc.tau_linear = 0; }
    for (int l = 0; l < N; ++l) if (p->kind[l] == HAP_MOE) dc.kindbits[l >> 6] |= 1ull << (l & 63);
    dc.kind_uniform_from = N - 1;
    while (dc.kind_uniform_from > 0 && p->kind[dc.kind_uniform_from - 1] == p->kind[N - 1]) --dc.kind_uniform_from;
    dc.kind_uniform = dc.kind_uniform_from == 0;
    dc.tab4 = p->d_tables;
    dc.tpre = dc.tab4 + 4 * n5; dc.tpost = dc.tpre + n4;

    guard.keep = true;
    *out = p;
    return HAP_OK;
}

// ------------------------------------------------------------------------------------------
// enumeration (host; at most a few thousand rows)
// ------------------------------------------------------------------------------------------
static uint64_t binom_sat(int n, int k, uint64_t sat)
{
    if (k < 0 || k > n) return 0;
    if (k > n - k) k = n - k;
    unsigned __int128 r = 1;
    for (int i = 1; i <= k; ++i) {
        r = r * (unsigned)(n - k + i) / (unsigned)i;
        if (r > sat) return sat;
    }
    return (uint64_t)r;
}

// distinct sequences with cnt[h] stages of type h: product of binomials, saturating
static uint64_t sequences_sat(const int *cnt, int T, uint64_t sat)
{
    int rem = 0;
    for (int h = 0; h < T; ++h) rem += cnt[h];
    unsigned __int128 r = 1;
    for (int h = 0; h < T; ++h) {
        r *= binom_sat(rem, cnt[h], sat);
        if (r > sat) return sat;
        rem -= cnt[h];
    }
    return (uint64_t)r;
}

// Prefix tree of the decoded mappings of one PP class (host copy `tab`: nmap x PP x (mask, link) bytes).
// A node is a distinct sequence of stage keys (types, link, load-balance window) of stages 1..d, d < PP;
// mappings that are consecutive in enumeration order share the nodes of their common prefix.  The window
// and the band of reachable end layers follow the same integer formulas as pipeline_dp_kernel; a node's
// band is the union over the mappings below it, which only adds cells that hold their plain recurrence
// value.  Returns false (and leaves the class on the general kernel) when the tree does not fit.
struct TriePartHost {
    TrieMeta meta;                          // device pointers are filled in after the upload
    std::vector<unsigned char> blob;        // nodes | leaves | cells | first_leaf | cell_gnode | parent | depth
    size_t o_nodes, o_leaves, o_cells, o_first, o_gnode, o_parent, o_depth;
    u32 n_nodes, n_cells, nmap, max_level;
    size_t smem;
};

// the tree of mappings [m0, m1) of the class
// `limit`: largest acceptable dynamic shared memory; a tree that needs more is abandoned before its records are written
static bool build_trie_part(hap_problem *p, const hap_problem::PpClass &cl, const uint8_t *tab_all, u64 m0, u64 m1, size_t limit,
                            TriePartHost &part)
{
    const int N = p->model.N, PP = cl.PP, T = p->T, R = p->prof.R;
    const u64 nmap = m1 - m0;
    const uint8_t *tab = tab_all + m0 * (u64)PP * 2;
    if (nmap == 0 || nmap > 65535) return false;
    struct Key { uint8_t mask, link, nmin, nmax; };
    struct HNode { u32 parent; Key k; int bl, bh; u32 first_leaf; };
    std::vector<std::vector<HNode>> lv(PP + 1);               // lv[d], d = 1..PP-1
    std::vector<TrieLeaf> leaves(nmap);
    std::vector<u32> path(PP + 1, 0);
    std::vector<Key> pkey(PP + 1);
    bool have_prev = false;
    i64 Pmin[1 << HAP_MAX_TYPES];
    for (int mk = 1; mk < (1 << T); ++mk) {
        i64 v = 0; bool seen = false;
        for (int h = 0; h < T; ++h) if (mk >> h & 1) { if (!seen || p->P[h] < v) v = p->P[h]; seen = true; }
        Pmin[mk] = v;
    }
    int capt_of[1 << HAP_MAX_TYPES] = {0};                      // type whose (smallest) memory binds a stage of these types
    for (int mk = 1; mk < (1 << T); ++mk) {
        i64 cap = 0; bool seen = false;
        for (int h = 0; h < T; ++h) if (mk >> h & 1) { if (!seen || p->cap_eff[h] < cap) { cap = p->cap_eff[h]; capt_of[mk] = h; } seen = true; }
    }
    const int delta_q = p->opts.delta_q;
    const bool uniform = (p->opts.flags & HAP_OPT_UNIFORM) != 0;
    std::vector<int> nmin(PP + 1), nmax(PP + 1), bl(PP + 1), bh(PP + 1);
    // the window of a stage depends on its type mask and on the mapping's summed compute power only: the two
    // divisions are done once per mask while that sum stays the same (it does for all sequences of a multiset)
    i64 win_Ps = -1;
    int win_lo[1 << HAP_MAX_TYPES], win_hi[1 << HAP_MAX_TYPES];
    for (u64 m = 0; m < nmap; ++m) {
        const uint8_t *row = tab + m * (u64)PP * 2;
        i64 Ps = 0;
        for (int s = 0; s < PP; ++s) {
            const int mk = row[s * 2];
            if (mk < 1 || mk >= (1 << T)) return false;
            Ps += Pmin[mk];
        }
        if (!uniform && delta_q >= 0 && Ps != win_Ps) {
            const i64 den = 1024 * Ps;
            for (int mk = 1; mk < (1 << T); ++mk) {
                i64 a = ((i64)(1024 - delta_q) * Pmin[mk] * N) / den;
                i64 b = ((i64)(1024 + delta_q) * Pmin[mk] * N + den - 1) / den;
                if (a < 1) a = 1;
                if (b > N - PP + 1) b = N - PP + 1;
                win_lo[mk] = (int)a; win_hi[mk] = (int)b;
            }
            win_Ps = Ps;
        }
        for (int s = 1; s <= PP; ++s) {
            int lo = 1, hi = N - PP + 1;
            if (uniform) { lo = N / PP; hi = (N + PP - 1) / PP; }
            else if (delta_q >= 0) { lo = win_lo[row[(s - 1) * 2]]; hi = win_hi[row[(s - 1) * 2]]; }
            if (lo < 0 || lo > 255 || hi < 0 || hi > 255) return false;
            nmin[s] = lo; nmax[s] = hi;
        }
        int tmin = 0, tmax = 0;
        for (int s = 1; s <= PP; ++s) { tmin += nmin[s]; tmax += nmax[s]; }
        bool dead = false;
        int smin = 0, smax = 0;
        for (int s = 1; s <= PP; ++s) {
            smin += nmin[s]; smax += nmax[s];
            int lo = smin > s ? smin : s, hi = smax < N - PP + s ? smax : N - PP + s;
            const int rl = N - (tmax - smax), rh = N - (tmin - smin);
            lo = lo > rl ? lo : rl; hi = hi < rh ? hi : rh;
            bl[s] = lo; bh[s] = hi;
            if (lo > hi) dead = true;
        }
        TrieLeaf &lf = leaves[m];
        std::memset(&lf, 0, sizeof(lf));
        lf.mask = row[(PP - 1) * 2]; lf.link = row[(PP - 1) * 2 + 1];
        lf.nmin = (uint8_t)nmin[PP]; lf.nmax = (uint8_t)nmax[PP];
        lf.dead = dead ? 1 : 0;
        lf.capt = (uint8_t)capt_of[lf.mask];
        if (dead) continue;
        int d0 = 1;                                              // first depth at which a new node is needed
        if (have_prev)
            for (; d0 < PP; ++d0) {
                const Key &k = pkey[d0];
                if (k.mask != row[(d0 - 1) * 2] || k.link != row[(d0 - 1) * 2 + 1] || k.nmin != nmin[d0] || k.nmax != nmax[d0]) break;
            }
        for (int d = d0; d < PP; ++d) {
            HNode nd;
            nd.parent = d > 1 ? path[d - 1] : 0;
            nd.k = Key{row[(d - 1) * 2], row[(d - 1) * 2 + 1], (uint8_t)nmin[d], (uint8_t)nmax[d]};
            nd.bl = 1 << 20; nd.bh = -1; nd.first_leaf = (u32)(m0 + m);
            pkey[d] = nd.k;
            path[d] = (u32)lv[d].size();
            lv[d].push_back(nd);
        }
        have_prev = true;
        for (int d = 1; d < PP; ++d) {
            HNode &nd = lv[d][path[d]];
            nd.bl = std::min(nd.bl, bl[d]); nd.bh = std::max(nd.bh, bh[d]);
        }
        lf.parent = PP > 1 ? (uint16_t)path[PP - 1] : 0;
    }
    // nodes of a depth ordered by the width of their window (widest first, stable), so that the cells a warp works
    // on have split loops of similar length
    for (int d = 1; d < PP; ++d) {
        std::vector<u32> ord(lv[d].size()), newidx(lv[d].size());
        for (size_t i = 0; i < ord.size(); ++i) ord[i] = (u32)i;
        std::stable_sort(ord.begin(), ord.end(), [&](u32 a, u32 b) {
            return (int)lv[d][a].k.nmax - (int)lv[d][a].k.nmin > (int)lv[d][b].k.nmax - (int)lv[d][b].k.nmin; });
        std::vector<HNode> sorted(lv[d].size());
        for (size_t i = 0; i < ord.size(); ++i) { sorted[i] = lv[d][ord[i]]; newidx[ord[i]] = (u32)i; }
        lv[d].swap(sorted);
        if (d + 1 < PP) for (auto &ch : lv[d + 1]) ch.parent = newidx[ch.parent];
        else for (u64 m = 0; m < nmap; ++m) if (!leaves[m].dead) leaves[m].parent = (uint16_t)newidx[leaves[m].parent];
    }
    // flat layout
    TrieMeta &tm = part.meta;
    std::memset(&tm, 0, sizeof(tm));
    tm.PP = PP; tm.nmap = (u32)nmap; tm.m_lo = (u32)m0;
    // row groups of the time rows: one per type mask that some stage has
    std::memset(tm.mrow_of, 255, sizeof(tm.mrow_of));
    {
        unsigned used = 0;
        for (int d = 1; d < PP; ++d) for (const auto &h : lv[d]) used |= 1u << h.k.mask;
        for (u64 m = 0; m < nmap; ++m) used |= 1u << leaves[m].mask;
        for (int mk = 1; mk < (1 << T); ++mk)
            if ((used >> mk) & 1u) { tm.mrow_of[mk] = (uint8_t)tm.n_mrows; tm.mask_of_row[tm.n_mrows] = (uint8_t)mk; tm.n_mrows++; }
    }
    u32 n_nodes = 0, n_cells = 0, max_level = 0;
    std::vector<std::vector<u32>> rowoff(PP + 1);
    for (int d = 1; d < PP; ++d) {
        if (lv[d].size() > 65535) return false;
        tm.node_lo[d] = n_nodes; tm.cell_lo[d] = n_cells;
        u32 c = 0;
        rowoff[d].resize(lv[d].size());
        for (size_t i = 0; i < lv[d].size(); ++i) { rowoff[d][i] = c; c += (u32)(lv[d][i].bh - lv[d][i].bl + 1); }
        tm.buf_cells[d & 1] = std::max(tm.buf_cells[d & 1], c);
        max_level = std::max(max_level, c);
        n_nodes += (u32)lv[d].size(); n_cells += c;
    }
    for (int d = std::max(PP, 1); d <= HAP_MAX_PP; ++d) { tm.node_lo[d] = n_nodes; tm.cell_lo[d] = n_cells; }
    {   // the shared memory the tree needs is known from the node bands: stop here if it is too much
        int widest = 1;
        for (int d = 1; d < PP; ++d) {
            int lo = 1 << 20, hi = -1;
            for (const auto &h : lv[d]) { lo = std::min(lo, h.bl); hi = std::max(hi, h.bh); }
            if (hi >= lo) widest = std::max(widest, hi - lo + 1);
        }
        const u32 be = (tm.buf_cells[0] + 1) / 2 * 2, bo = (tm.buf_cells[1] + 1) / 2 * 2;
        part.smem = trie_smem_bytes(N, PP, T, R, tm.n_mrows, p->dc.kind_uniform ? 1 : widest, be, bo, n_cells, n_nodes);
        if (part.smem > limit) return false;
    }
    tm.buf_cells[0] = (tm.buf_cells[0] + 1) / 2 * 2; tm.buf_cells[1] = (tm.buf_cells[1] + 1) / 2 * 2;
    if (n_cells >= (1u << 25)) return false;
    std::vector<TrieNode> nodes(n_nodes);
    std::vector<uint16_t> parent(n_nodes);
    std::vector<TrieCell> cells(n_cells);
    std::vector<u32> cell_gnode(n_cells);
    int band_max = 1;
    for (int d = 1; d <= PP; ++d) { tm.jlo[d] = 255; tm.jhi[d] = 0; tm.wmax[d] = 0; tm.tmask[d] = 0; tm.kmin[d] = 255; tm.kmax[d] = 0; }
    tm.jlo[PP] = tm.jhi[PP] = (uint8_t)N;
    for (u64 m = 0; m < nmap; ++m) {
        if (leaves[m].dead) continue;
        tm.wmax[PP] = std::max(tm.wmax[PP], leaves[m].nmax);
        tm.tmask[PP] |= (uint8_t)(1u << leaves[m].capt);
    }
    std::vector<u32> first_leaf(n_nodes);
    std::vector<uint8_t> depth(n_nodes);
    for (int d = 1; d < PP; ++d) {
        // per-depth extremes are gathered in locals (the description's byte fields alias everything the loop writes)
        int d_jlo = 255, d_jhi = 0, d_wmax = 0, d_kmin = 255, d_kmax = 0;
        unsigned d_tmask = 0;
        const u32 node_lo = tm.node_lo[d], cell_lo = tm.cell_lo[d];
        const u32 *ro = rowoff[d].data();
        TrieCell *cd = cells.data();
        u32 *gn = cell_gnode.data();
        for (size_t i = 0; i < lv[d].size(); ++i) {
            const HNode &h = lv[d][i];
            TrieNode nd{};
            nd.rowoff = ro[i];
            nd.mask = h.k.mask; nd.link = h.k.link; nd.nmin = h.k.nmin; nd.nmax = h.k.nmax;
            nd.bl = (uint8_t)h.bl; nd.bh = (uint8_t)h.bh;
            if (d > 1) { const HNode &ph = lv[d - 1][h.parent]; nd.prowoff = rowoff[d - 1][h.parent]; nd.pbl = (uint8_t)ph.bl; nd.pbh = (uint8_t)ph.bh; }
            else { nd.prowoff = 0; nd.pbl = 0; nd.pbh = 0; }
            nodes[node_lo + i] = nd;
            parent[node_lo + i] = (uint16_t)h.parent;
            first_leaf[node_lo + i] = h.first_leaf;
            depth[node_lo + i] = (uint8_t)d;
            d_jlo = std::min<int>(d_jlo, nd.bl); d_jhi = std::max<int>(d_jhi, nd.bh);
            d_wmax = std::max<int>(d_wmax, nd.nmax);
            d_tmask |= 1u << capt_of[nd.mask];
            const int cls = nd.link & 3, ha = (nd.link >> 2) & 3, hb = (nd.link >> 4) & 3;
            const u32 kidx = d == 1 ? tm.mrow_of[nd.mask] : 16 + hb * 6 + (cls == HAP_CROSS ? 2 + ha : cls);
            const u32 cx = (u32)((int)nd.prowoff - (int)nd.pbl + 256) | (kidx << 26);
            const u32 cw = (u32)tm.mrow_of[nd.mask] * (u32)(R * (N + 1));
            const u32 g = node_lo + (u32)i;
            const int nmx = nd.nmax, nmn = nd.nmin, pbl = nd.pbl, pbh = nd.pbh;
            u32 c = cell_lo + ro[i];
            for (int j = h.bl; j <= h.bh; ++j, ++c) {
                int klo = std::max(j - nmx, pbl), khi = std::min(j - nmn, pbh);
                if (klo > khi) { klo = 1; khi = 0; }
                else { d_kmin = std::min(d_kmin, klo); d_kmax = std::max(d_kmax, khi); }
                TrieCell cc;
                cc.x = cx;
                cc.y = (u32)j | ((u32)klo << 8) | ((u32)khi << 16);
                cc.z = 0;                                         // threshold index: needs the depth's first end layer, set below
                cc.w = cw;
                cd[c] = cc;
                gn[c] = g;
            }
        }
        tm.jlo[d] = (uint8_t)d_jlo; tm.jhi[d] = (uint8_t)d_jhi; tm.wmax[d] = (uint8_t)d_wmax;
        tm.tmask[d] = (uint8_t)d_tmask; tm.kmin[d] = (uint8_t)d_kmin; tm.kmax[d] = (uint8_t)d_kmax;
    }
    for (int d = 1; d <= PP; ++d) if (tm.jlo[d] <= tm.jhi[d]) band_max = std::max(band_max, tm.jhi[d] - tm.jlo[d] + 1);
    for (u64 m = 0; m < nmap; ++m) {
        TrieLeaf &lf = leaves[m];
        if (lf.dead || PP == 1) { lf.prowoff = 0; lf.pbl = 0; lf.pbh = 0; continue; }
        const HNode &ph = lv[PP - 1][lf.parent];
        lf.prowoff = rowoff[PP - 1][lf.parent]; lf.pbl = (uint8_t)ph.bl; lf.pbh = (uint8_t)ph.bh;
    }
    for (u64 m = 0; m < nmap; ++m) {
        const TrieLeaf &lf = leaves[m];
        if (lf.dead) continue;
        const int klo = std::max(N - (int)lf.nmax, (int)lf.pbl), khi = std::min(N - (int)lf.nmin, (int)lf.pbh);
        if (klo <= khi) { tm.kmin[PP] = std::min<uint8_t>(tm.kmin[PP], (uint8_t)klo); tm.kmax[PP] = std::max<uint8_t>(tm.kmax[PP], (uint8_t)khi); }
    }
    // A depth whose cells only look at splits behind the last change of layer kind sees spans of one kind only:
    // their memory depends on the length alone and a threshold row of that depth is one number.  All depths of a
    // model whose layers are all of one kind; every depth but the first few of a model with a dense prefix.
    bool all_flat = true;
    for (int d = 1; d <= PP; ++d) {
        tm.flat[d] = (tm.kmin[d] > tm.kmax[d] || (int)tm.kmin[d] >= p->dc.kind_uniform_from) ? 1 : 0;
        all_flat = all_flat && tm.flat[d];
    }
    tm.all_flat = all_flat ? 1 : 0;
    const int thr_w = all_flat ? 1 : band_max;
    tm.thr_w = thr_w;
    for (u32 c = 0; c < n_cells; ++c) {
        const u32 g = cell_gnode[c];
        const int d = depth[g], j = (int)(cells[c].y & 255);
        cells[c].z = (u32)((((d - 1) * T + capt_of[nodes[g].mask]) * R) * thr_w + ((thr_w == 1 || tm.flat[d]) ? 0 : j - (int)tm.jlo[d]));
    }
    tm.band_max = band_max;
    const size_t smem = trie_smem_bytes(N, PP, T, R, tm.n_mrows, thr_w, tm.buf_cells[0], tm.buf_cells[1], n_cells, n_nodes);
    if (smem > limit) return false;
    // one blob: nodes | leaves | cells | first_leaf | cell_gnode | parent | depth
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    part.o_nodes = 0; part.o_leaves = up(part.o_nodes + (size_t)n_nodes * sizeof(TrieNode));
    part.o_cells = up(part.o_leaves + nmap * sizeof(TrieLeaf));
    part.o_first = up(part.o_cells + (size_t)n_cells * sizeof(TrieCell)); part.o_gnode = up(part.o_first + (size_t)n_nodes * 4);
    part.o_parent = up(part.o_gnode + (size_t)n_cells * 4); part.o_depth = up(part.o_parent + (size_t)n_nodes * 2);
    const size_t total = up(part.o_depth + n_nodes) + 256;
    part.blob.assign(total, 0);
    unsigned char *blob = part.blob.data();
    if (n_nodes) std::memcpy(blob + part.o_nodes, nodes.data(), (size_t)n_nodes * sizeof(TrieNode));
    std::memcpy(blob + part.o_leaves, leaves.data(), nmap * sizeof(TrieLeaf));
    if (n_cells) std::memcpy(blob + part.o_cells, cells.data(), (size_t)n_cells * sizeof(TrieCell));
    if (n_nodes) std::memcpy(blob + part.o_first, first_leaf.data(), (size_t)n_nodes * 4);
    if (n_cells) std::memcpy(blob + part.o_gnode, cell_gnode.data(), (size_t)n_cells * 4);
    if (n_nodes) std::memcpy(blob + part.o_parent, parent.data(), (size_t)n_nodes * 2);
    if (n_nodes) std::memcpy(blob + part.o_depth, depth.data(), n_nodes);
    part.n_nodes = n_nodes; part.n_cells = n_cells; part.nmap = (u32)nmap; part.max_level = max_level; part.smem = smem;
    return true;
}

// Builds the class's tree, as one part or, when one part would leave room for only one block per SM, as up to
// eight parts over contiguous ranges of mappings (the few nodes near the root that two parts share are computed by
// both).  Returns false (the class stays on the general kernel) when nothing fits.
struct TrieClassHost { std::vector<TriePartHost> parts; unsigned masks_used = 0xffffffffu; };
// what upload_tries gets per class: the class, its (shared) host tree and the class's configurations
struct TrieBuilt { hap_problem::PpClass *cl; std::shared_ptr<const TrieClassHost> tree; std::vector<u32> plist; };

static bool build_trie(hap_problem *p, hap_problem::PpClass &cl, const uint8_t *tab, u64 nmap, size_t n_conf, TrieClassHost &out)
{
    if (nmap == 0 || n_conf == 0) return false;
    constexpr size_t kTwoPerSm = 108 * 1024;                 // dynamic shared memory that lets two blocks share an SM
    const size_t slots = (cl.item_hi - cl.item_lo) / n_conf;             // work items per configuration
    std::vector<TriePartHost> parts;
    // The number of parts that worked for a class of this shape before is tried first (a hint kept per process: a
    // wrong hint costs one failed attempt, the sequence below then runs as usual).
    static std::mutex hint_mu;
    static std::map<std::array<long long, 6>, int> hint;
    const std::array<long long, 6> key = {cl.PP, (long long)nmap, p->model.N, p->T * 16 + p->prof.R, p->opts.delta_q, (long long)(p->opts.flags & HAP_OPT_UNIFORM)};
    int first_np = 0;
    { std::lock_guard<std::mutex> lock(hint_mu); auto it = hint.find(key); if (it != hint.end()) first_np = it->second; }
    auto attempt = [&](int np) {
        if ((u64)np > nmap || (np > 1 && (size_t)np > slots)) return false;
        std::vector<TriePartHost> cand(np);
        bool ok = true;
        for (int q = 0; q < np && ok; ++q) ok = build_trie_part(p, cl, tab, nmap * q / np, nmap * (q + 1) / np, kTwoPerSm, cand[q]);
        if (ok) parts.swap(cand);
        return ok;
    };
    int used_np = 0;
    if (first_np > 1 && attempt(first_np)) used_np = first_np;
    if (!used_np)
        for (int np : {1, 2, 3, 4, 6, 8}) {
            if ((u64)np > nmap || (np > 1 && (size_t)np > slots)) break;
            if (np == first_np) continue;
            if (attempt(np)) { used_np = np; break; }
        }
    if (used_np) { std::lock_guard<std::mutex> lock(hint_mu); hint[key] = used_np; }
    if (parts.empty()) {                                     // no split lets two blocks share an SM: one block per SM
        parts.resize(1);
        if (!build_trie_part(p, cl, tab, 0, nmap, 220 * 1024, parts[0])) parts.clear();
    }
    if (parts.empty()) return false;
    out.parts.swap(parts);
    return true;
}

// One allocation for the trees of all classes.  Its head holds what does not depend on where it lies -- per class the
// parts' blobs and the list of the class's configurations -- and is copied from an image kept per process under
// `image_key` (the classes' tree keys and the enumeration's key); behind it lie the part descriptions and the job
// list of the gather kernel, which hold device addresses and are staged for every problem.
namespace {
std::mutex g_tree_image_mu;
std::map<std::string, std::shared_ptr<PinnedImage>> g_tree_images;
constexpr size_t kTreeImages = 16;
}

static bool upload_tries(hap_problem *p, std::vector<TrieBuilt> &built, const std::string &image_key)
{
    constexpr size_t kTwoPerSm = 108 * 1024;
    auto up = [](size_t v) { return (v + 255) / 256 * 256; };
    size_t head = 0, tail = 0, n_parts_all = 0;
    for (auto &bc : built) {
        for (const auto &pt : bc.tree->parts) head += up(pt.blob.size());
        head += up(bc.plist.size() * sizeof(u32));
        tail += up(bc.tree->parts.size() * sizeof(TrieMeta));
        n_parts_all += bc.tree->parts.size();
    }
    if (!head) return true;
    const size_t o_jobs = head + tail;
    const size_t total = o_jobs + up(n_parts_all * sizeof(GatherJob));
    std::vector<GatherJob> gjobs;
    DecodeJobs dj{};
    unsigned dblk = 0, gblk = 0;
    if (cached_malloc(p->device, (void **)&p->d_trie_arena, total) != cudaSuccess) { p->d_trie_arena = nullptr; cudaGetLastError(); return false; }
    // the head: blobs and configuration lists (`stage` may be null: only the offsets are wanted then)
    auto fill_head = [&](unsigned char *stage) {
        size_t off = 0;
        for (auto &bc : built) {
            for (const auto &pt : bc.tree->parts) {
                if (stage) std::memcpy(stage + off, pt.blob.data(), pt.blob.size());
                off += up(pt.blob.size());
            }
            if (stage) std::memcpy(stage + off, bc.plist.data(), bc.plist.size() * sizeof(u32));
            off += up(bc.plist.size() * sizeof(u32));
        }
    };
    // the tail: part descriptions and gather jobs, with this arena's addresses; also fills the per-class records
    auto fill_tail = [&](unsigned char *stage) -> bool {          // (stage = start of the tail)
    size_t off = 0, toff = 0;
    for (auto &bc : built) {
        hap_problem::Trie &tr = bc.cl->trie;
        const TrieClassHost &h = *bc.tree;
        std::vector<TrieMeta> metas;
        size_t smem = 0;
        u32 want = 0;
        for (const auto &pt : h.parts) {
            unsigned char *base = p->d_trie_arena + off;
            hap_problem::TriePartDev pd{};
            pd.d_nodes = reinterpret_cast<TrieNode *>(base + pt.o_nodes);
            pd.d_leaves = reinterpret_cast<TrieLeaf *>(base + pt.o_leaves);
            pd.d_cells = reinterpret_cast<TrieCell *>(base + pt.o_cells);
            pd.d_first_leaf = reinterpret_cast<u32 *>(base + pt.o_first);
            pd.d_gnode = reinterpret_cast<u32 *>(base + pt.o_gnode);
            pd.d_depth = base + pt.o_depth;
            pd.n_nodes = pt.n_nodes; pd.n_cells = pt.n_cells; pd.nmap = pt.nmap; pd.m_lo = pt.meta.m_lo;
            std::memcpy(pd.mrow_of, pt.meta.mrow_of, sizeof(pd.mrow_of));
            TrieMeta meta = pt.meta;                 // the host tree is shared between problems: the device pointers go into a copy
            meta.nodes = pd.d_nodes; meta.leaves = pd.d_leaves; meta.cells = pd.d_cells;
            meta.parent = reinterpret_cast<const uint16_t *>(base + pt.o_parent);
            tr.parts.push_back(pd);
            metas.push_back(meta);
            GatherJob gj{};
            gj.first_leaf = pd.d_first_leaf; gj.gnode = pd.d_gnode; gj.depth = pd.d_depth;
            gj.nodes = pd.d_nodes; gj.cells = pd.d_cells; gj.leaves = pd.d_leaves;
            gj.tab_off = bc.cl->map_base; gj.n_nodes = pd.n_nodes; gj.n_cells = pd.n_cells; gj.nmap = pd.nmap; gj.m_lo = pd.m_lo;
            gj.blk_lo = gblk; gj.PP = bc.cl->PP;
            std::memcpy(gj.rm.mrow_of, pd.mrow_of, sizeof(gj.rm.mrow_of));
            gblk += (pd.n_nodes + pd.n_cells + pd.nmap + 255) / 256;
            gjobs.push_back(gj);
            smem = std::max(smem, pt.smem);
            want = std::max(want, std::max(pt.max_level, pt.nmap));
            off += up(pt.blob.size());
        }
        tr.d_plist = reinterpret_cast<u32 *>(p->d_trie_arena + off);
        off += up(bc.plist.size() * sizeof(u32));
        tr.d_metas = reinterpret_cast<TrieMeta *>(p->d_trie_arena + head + toff);
        std::memcpy(stage + toff, metas.data(), metas.size() * sizeof(TrieMeta));
        toff += up(metas.size() * sizeof(TrieMeta));
        tr.n_conf = (unsigned)bc.plist.size(); tr.smem = smem;
        if (dj.n <= HAP_MAX_PP) {
            const hap_problem::PpClass &cl = *bc.cl;
            const u32 rep = p->items[cl.item_lo].p;
            const u64 nmap_cl = p->pconfs[rep].nmap;
            dj.blk_lo[dj.n] = dblk; dj.p_rep[dj.n] = rep; dj.nmap[dj.n] = (u32)nmap_cl; dj.tab_off[dj.n] = cl.map_base;
            dblk += (unsigned)((nmap_cl + 3) / 4);
            dj.n++;
            dj.blk_lo[dj.n] = dblk;
        }
        // a thread takes about four cells of the widest depth (measured: smaller blocks, more of them per SM)
        const int th = (int)(((want + 3) / 4 + 31) / 32 * 32);
        tr.threads = std::min(smem <= kTwoPerSm ? 512 : 1024, std::max(128, th));
        tr.ok = true;
    }
    std::memcpy(stage + tail, gjobs.data(), gjobs.size() * sizeof(GatherJob));
    return true;
    };
    // head: from the process's image of these trees when there is one (made on first use)
    std::shared_ptr<PinnedImage> image;
    if (upload_stream(p->device)) {
        std::lock_guard<std::mutex> lock(g_tree_image_mu);
        auto it = g_tree_images.find(image_key);
        if (it != g_tree_images.end() && it->second->bytes == head) image = it->second;
        else if ((image = pinned_image(head))) {
            std::memset(image->ptr, 0, head);
            fill_head(static_cast<unsigned char *>(image->ptr));
            if (g_tree_images.size() >= kTreeImages) g_tree_images.clear();
            g_tree_images[image_key] = image;
        }
    }
    cudaError_t e = image ? upload_image(p, p->d_trie_arena, *image, head)
                          : upload(p, p->d_trie_arena, head, [&](unsigned char *stage) { fill_head(stage); return true; });
    if (e == cudaSuccess) e = upload(p, p->d_trie_arena + head, total - head, fill_tail);
    if (e != cudaSuccess) {
        cudaGetLastError();
        for (auto &bc : built) bc.cl->trie = hap_problem::Trie{};
        return false;
    }
    p->tree_image = image;
    p->decode_jobs = dj;
    p->d_gather_jobs = reinterpret_cast<GatherJob *>(p->d_trie_arena + o_jobs);
    p->n_gather_jobs = (int)gjobs.size();
    p->gather_blocks = gblk;
    return true;
}

// ---- per-process cache of the classes' prefix trees ------------------------------------------------------
namespace {
std::mutex g_trie_cache_mu;
std::map<std::string, std::shared_ptr<const TrieClassHost>> g_trie_cache;
constexpr size_t kTrieCacheEntries = 256;
}

template <class V> static void key_put(std::string &k, const V &v) { k.append(reinterpret_cast<const char *>(&v), sizeof(v)); }

// everything the decoded mappings, the windows, the bands, the cell records and the split into parts depend on
static std::string trie_cache_key(const hap_problem *p, const hap_problem::PpClass &cl)
{
    std::string k("hap-trie-1");
    const hap_pconf &rep = p->pconfs[p->items[cl.item_lo].p];
    const size_t n_conf = p->items[cl.item_hi - 1].p - p->items[cl.item_lo].p + 1;
    const int32_t head[] = {p->model.N, p->T, p->prof.R, cl.PP, rep.G, rep.mode, p->opts.delta_q, (int32_t)(p->opts.flags & HAP_OPT_UNIFORM),
                            p->dc.kind_uniform, p->dc.kind_uniform_from, (int32_t)((cl.item_hi - cl.item_lo) / n_conf)};
    key_put(k, head);
    key_put(k, rep.nmap);
    for (int h = 0; h < p->T; ++h) { key_put(k, p->P[h]); key_put(k, p->cap_eff[h]); key_put(k, p->dc.m[h]); key_put(k, p->dc.node_size[h]); }
    return k;
}

static std::shared_ptr<const TrieClassHost> trie_cache_find(const std::string &key)
{
    std::lock_guard<std::mutex> lock(g_trie_cache_mu);
    auto it = g_trie_cache.find(key);
    return it == g_trie_cache.end() ? nullptr : it->second;
}

static void trie_cache_insert(const std::string &key, std::shared_ptr<const TrieClassHost> tree)
{
    std::lock_guard<std::mutex> lock(g_trie_cache_mu);
    if (g_trie_cache.size() >= kTrieCacheEntries) g_trie_cache.clear();
    g_trie_cache[key] = std::move(tree);
}

// the configurations of a class (contiguous: PP is the outermost loop of the enumeration)
static std::vector<u32> class_plist(const hap_problem *p, const hap_problem::PpClass &cl)
{
    std::vector<u32> plist;
    for (size_t pi = p->items[cl.item_lo].p; pi <= p->items[cl.item_hi - 1].p; ++pi) plist.push_back((u32)pi);
    return plist;
}

// ---- per-process cache of enumerations -----------------------------------------------------------------------
struct EnumResult {
    std::vector<hap_pconf> rows;
    std::vector<WorkItem> items;
    std::vector<hap_problem::PpClass> classes;       // streams, events and trees are per problem: empty here
    uint64_t n_cand = 0;
    u64 tab_bytes = 0;
    std::shared_ptr<PinnedImage> image;             // rows | padding to 256 bytes | items | padding: the head of a problem's arena (may be null)
};
namespace {
std::mutex g_enum_cache_mu;
std::map<std::string, std::shared_ptr<const EnumResult>> g_enum_cache;
constexpr size_t kEnumCacheEntries = 64;
}

// every input of the enumeration loop nest and of the block shapes of the classes
static std::string enum_cache_key(const hap_problem *p)
{
    std::string k("hap-enum-1");
    const hap_model &mo = p->model;
    const int64_t head[] = {mo.N, mo.S, mo.E, mo.GB, mo.nq, mo.nkv, p->T, p->W, p->prof.R, p->dc.tau_linear, p->opts.tp_max,
                            p->opts.n_rc, (int64_t)p->opts.map_cap, (int64_t)(p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT | HAP_OPT_NO_MAPTAB))};
    key_put(k, head);
    for (int h = 0; h < p->T; ++h) key_put(k, p->m[h]);
    auto put_list = [&](const std::vector<int> &v) { const int64_t n = (int64_t)v.size(); key_put(k, n); for (int x : v) key_put(k, x); };
    put_list(p->pp_list); put_list(p->tp_list); put_list(p->cp_list); put_list(p->ep_list); put_list(p->tpe_list); put_list(p->mb_list);
    return k;
}

static std::shared_ptr<const EnumResult> enum_cache_find(const std::string &key)
{
    std::lock_guard<std::mutex> lock(g_enum_cache_mu);
    auto it = g_enum_cache.find(key);
    return it == g_enum_cache.end() ? nullptr : it->second;
}

static void enum_cache_insert(const std::string &key, std::shared_ptr<const EnumResult> r)
{
    std::lock_guard<std::mutex> lock(g_enum_cache_mu);
    if (g_enum_cache.size() >= kEnumCacheEntries) g_enum_cache.clear();
    g_enum_cache[key] = std::move(r);
}

extern "C" hap_status hap_enumerate(hap_problem *p, uint64_t *n_pconf, uint64_t *n_candidates)
{
    if (!p) return HAP_E_INVALID;
    if (cudaSetDevice(p->device) != cudaSuccess) return fail(p, HAP_E_CUDA, "cudaSetDevice");
    if (!p->enumerated) {
        const hap_model &mo = p->model;
        const int N = mo.N, T = p->T;
        // The configuration table, the work items and the PP classes are a function of the model's dimensions, the
        // cluster inventory and the search options -- not of the profiled tables: they are kept per process, so that
        // planning again for the same cluster and lists copies them instead of running the loop nest.
        const std::string ekey = enum_cache_key(p);
        std::shared_ptr<const EnumResult> er = enum_cache_find(ekey);
        if (!er) {
            auto fresh = std::make_shared<EnumResult>();
            hap_status es = [&]() -> hap_status {
        std::vector<hap_pconf> rows;
            rows.reserve(p->pp_list.size() * p->tp_list.size() * p->cp_list.size() * p->ep_list.size() * p->tpe_list.size() * p->mb_list.size() / 4 + 16);
            uint64_t off = 0;
            const uint64_t SAT = 1ull << 62;
            for (int PP : p->pp_list) {
                if (PP > N || PP > HAP_MAX_PP || p->W % PP) continue;
                const int64_t G = p->W / PP;
                if (G > 0x7fffffffll) continue;
                bool homog = true;
                int cnt[HAP_MAX_TYPES] = {0, 0, 0, 0};
                for (int h = 0; h < T; ++h) { if (p->m[h] % G) homog = false; cnt[h] = (int)(p->m[h] / G); }
                const uint64_t nms = homog ? sequences_sat(cnt, T, SAT) : 0;
                const int mode = (homog && nms <= p->opts.map_cap) ? HAP_MAP_MULTISET : HAP_MAP_BLOCK;
                uint64_t nmap = nms;
                if (mode == HAP_MAP_BLOCK) { nmap = 1; for (int i = 2; i <= T; ++i) nmap *= (uint64_t)i; }
                for (int itp = 0; itp < (int)p->tp_list.size(); ++itp) {
                    const int TP = p->tp_list[itp];
                    if (G % TP || TP > p->opts.tp_max || mo.nq % TP || mo.nkv % TP) continue;
                    for (int icp = 0; icp < (int)p->cp_list.size(); ++icp) {
                        const int CP = p->cp_list[icp];
                        if (G % ((int64_t)TP * CP) || mo.S % (2 * CP)) continue;
                        const int64_t DP = G / ((int64_t)TP * CP);
                        for (int iep = 0; iep < (int)p->ep_list.size(); ++iep) {
                            const int EP = p->ep_list[iep];
                            if (mo.E % EP || G % EP) continue;
                            for (int TPE : p->tpe_list) {
                                if (G % ((int64_t)EP * TPE) || TPE > p->opts.tp_max) continue;
                                const int64_t EDP = G / ((int64_t)EP * TPE);
                                for (int ib = 0; ib < (int)p->mb_list.size(); ++ib) {
                                    const int b = p->mb_list[ib];
                                    if (mo.GB % (DP * b)) continue;
                                    hap_pconf q{};
                                    q.PP = PP; q.TP = TP; q.CP = CP; q.DP = (int)DP; q.EP = EP; q.TPE = TPE; q.b = b;
                                    q.M = (int)(mo.GB / (DP * b)); q.EDP = (int)EDP; q.G = (int)G;
                                    q.itp = itp; q.icp = icp; q.ib = ib; q.iep = iep; q.mode = mode; q.reserved = 0;
                                    q.nmap = nmap; q.offset = off;
                                    if (nmap > (SAT - off) / (uint64_t)p->opts.n_rc) return fail(p, HAP_E_RANGE, "candidate space overflows 2^62");
                                    off += nmap * (uint64_t)p->opts.n_rc;
                                    rows.push_back(q);
                                }
                            }
                        }
                    }
                }
            }
            if (rows.empty()) return fail(p, HAP_E_INFEASIBLE, "no parallel configuration divides the cluster");
            if (rows.size() > 0xffffffffull) return fail(p, HAP_E_RANGE, "too many configurations");

            // PP classes (heaviest first).  Each class is one launch with its own block shape; a class keeps a
            // table of its decoded mappings when that table is small.
            std::vector<int> pps;
            for (const auto &r : rows) if (std::find(pps.begin(), pps.end(), r.PP) == pps.end()) pps.push_back(r.PP);
            std::sort(pps.begin(), pps.end(), [](int a, int b) { return a > b; });
            std::vector<WorkItem> items;
            items.reserve(rows.size() * 2);
            std::vector<hap_problem::PpClass> classes;
            u64 tab_bytes = 0;
            for (int PP : pps) {
                hap_problem::PpClass cl{};
                cl.PP = PP;
                cl.masks_used = 0xffffffffu;
                cl.stream = nullptr; cl.done = nullptr;
                cl.warps = 0;
                // the rows of a PP value are contiguous (PP is the outermost loop of the enumeration)
                size_t row_lo = 0;
                while (row_lo < rows.size() && rows[row_lo].PP != PP) ++row_lo;
                size_t row_hi = row_lo;
                while (row_hi < rows.size() && rows[row_hi].PP == PP) ++row_hi;
                cl.multiset = rows[row_lo].mode == HAP_MAP_MULTISET;
                // most warps per SM: try block shapes from large to small, keep the one with the most resident warps
                int best_resident = 0;
                const uint64_t class_nmap = rows[row_lo].nmap;
                const uint64_t per_pconf = class_nmap * (uint64_t)p->opts.n_rc;     // candidates a block can have at most
                for (int w : {12, 8, 6, 4, 2, 1}) {
                    if ((uint64_t)w * 8 > per_pconf && w > 2) continue;             // keep about 8 candidates per warp
                    const size_t sm = dp_smem_bytes(N, PP, T, p->prof.R, w, cl.multiset, p->dc.tau_linear != 0,
                                                    (p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT)) != 0);
                    if (sm > 227 * 1024) continue;
                    const int per_sm = std::min<int>((int)((227 * 1024) / (sm + 1024)), std::min(32, 64 / w));
                    const int resident = std::min(per_sm * w, 24);           // registers allow about 24 warps per SM
                    if (resident > best_resident) { best_resident = resident; cl.warps = w; cl.smem = sm; }
                }
                if (!cl.warps) return fail(p, HAP_E_RANGE, "shared memory need of a PP=%d block exceeds the SM", PP);
                // a warp takes a slice of at most 64 consecutive mappings (one bit each in its infeasibility masks)
                const uint64_t chunk_cap = 32ull * cl.warps;
                cl.item_lo = items.size();
                uint64_t nmap = 0;
                for (size_t pi = row_lo; pi < row_hi; ++pi) {
                    nmap = rows[pi].nmap;
                    const uint64_t n_chunks = (nmap + chunk_cap - 1) / chunk_cap;
                    const uint64_t chunk = (nmap + n_chunks - 1) / n_chunks;          // balanced chunks
                    for (uint64_t lo = 0; lo < nmap; lo += chunk) {
                        WorkItem it; it.p = (uint32_t)pi; it.lo = lo; it.count = (uint32_t)std::min<uint64_t>(chunk, nmap - lo);
                        items.push_back(it);
                    }
                }
                cl.item_hi = items.size();
                cl.has_tab = !(p->opts.flags & HAP_OPT_NO_MAPTAB) && nmap * (uint64_t)PP * 2 <= (64ull << 20) &&
                             tab_bytes + nmap * PP * 2 <= (256ull << 20);
                cl.map_base = tab_bytes;
                if (cl.has_tab) tab_bytes += (nmap * (uint64_t)PP * 2 + 255) / 256 * 256;
                classes.push_back(cl);
            }
            if (items.size() > 0x7fffffffull) return fail(p, HAP_E_RANGE, "too many work items");

            fresh->rows.swap(rows); fresh->items.swap(items); fresh->classes.swap(classes);
            fresh->n_cand = off; fresh->tab_bytes = tab_bytes;
            {   // the table and the items as every problem with these lists uploads them
                auto up = [](size_t v) { return (v + 255) / 256 * 256; };
                const size_t o_items = up(fresh->rows.size() * sizeof(hap_pconf)), total = up(o_items + fresh->items.size() * sizeof(WorkItem));
                fresh->image = pinned_image(total);
                if (fresh->image) {
                    unsigned char *im = static_cast<unsigned char *>(fresh->image->ptr);
                    std::memset(im, 0, total);
                    std::memcpy(im, fresh->rows.data(), fresh->rows.size() * sizeof(hap_pconf));
                    std::memcpy(im + o_items, fresh->items.data(), fresh->items.size() * sizeof(WorkItem));
                }
            }
            return HAP_OK;
            }();
            if (es != HAP_OK) return es;
            enum_cache_insert(ekey, fresh);
            er = fresh;
        }
        p->enum_ref = er;
        p->pconfs.ptr = er->rows.data(); p->pconfs.n = er->rows.size();
        p->items.ptr = er->items.data(); p->items.n = er->items.size();
        p->classes = er->classes;
        const uint64_t off = er->n_cand;
        const u64 tab_bytes = er->tab_bytes;
        p->n_cand = off;
        const size_t np = p->pconfs.size();
        // one allocation for everything whose size the enumeration fixes (an allocation costs far more than the
        // microseconds a pass takes): configuration table | work items | layer costs | coefficients | per-type
        // constants | lower bounds | partial minima | mapping tables | small scalars
        // partial minima of a search: one slot per block; a class's tree kernel may run up to 8 parts per configuration
        // (the exact count is fixed below, once the trees are built)
        p->n_partial = 1024;
        for (const auto &cl : p->classes) {
            const size_t n_conf = p->items[cl.item_hi - 1].p - p->items[cl.item_lo].p + 1;
            p->n_partial += std::max(cl.item_hi - cl.item_lo, n_conf * 8);
        }
        {
            auto up = [](size_t v) { return (v + 255) / 256 * 256; };
            size_t o = 0;
            const size_t o_pconf = o; o = up(o + np * sizeof(hap_pconf));
            const size_t o_items = o; o = up(o + p->items.size() * sizeof(WorkItem));
            const size_t o_c2 = o; o = up(o + np * T * N * 2 * sizeof(i64));
            const size_t o_coef = o; o = up(o + np * T * HAP_NCOEF * sizeof(i64));
            const size_t o_tc = o; o = up(o + np * T * sizeof(TypeConst));
            const size_t o_lb = o; o = up(o + np * sizeof(i64));
            const size_t o_pcost = o; o = up(o + p->n_partial * sizeof(i64));
            const size_t o_pindex = o; o = up(o + p->n_partial * sizeof(u64));
            const size_t o_maptab = o; o = up(o + tab_bytes);
            const size_t o_range = o; o = up(o + sizeof(u64));
            const size_t o_counters = o; o = up(o + 8 * sizeof(u64));
            const size_t o_best = o; o = up(o + 2 * sizeof(i64));
            const size_t o_single = o; o = up(o + sizeof(SingleOut));
            CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_arena, o));
            unsigned char *base = p->d_arena;
            p->d_pconf = reinterpret_cast<hap_pconf *>(base + o_pconf); p->d_items = reinterpret_cast<WorkItem *>(base + o_items);
            p->d_c2 = reinterpret_cast<i64 *>(base + o_c2); p->d_coef = reinterpret_cast<i64 *>(base + o_coef);
            p->d_tc = reinterpret_cast<TypeConst *>(base + o_tc); p->d_lb = reinterpret_cast<i64 *>(base + o_lb);
            p->d_pcost = reinterpret_cast<i64 *>(base + o_pcost); p->d_pindex = reinterpret_cast<u64 *>(base + o_pindex);
            p->d_maptab = tab_bytes ? base + o_maptab : nullptr;
            p->d_range = reinterpret_cast<u64 *>(base + o_range); p->d_counters = reinterpret_cast<u64 *>(base + o_counters);
            p->d_best = reinterpret_cast<i64 *>(base + o_best); p->d_single = base + o_single;
            // configuration table and work items travel in one copy (they are adjacent up to padding)
            if (er->image && er->image->bytes == o_c2) CUDA_TRY(p, upload_image(p, base, *er->image, o_c2));
            else CUDA_TRY(p, upload(p, base, o_c2, [&](unsigned char *stage) {
                std::memcpy(stage + o_pconf, p->pconfs.data(), np * sizeof(hap_pconf));
                std::memcpy(stage + o_items, p->items.data(), p->items.size() * sizeof(WorkItem));
                return true; }));
            if (p->upload_pending) {
                cudaStream_t us = upload_stream(p->device);
                CUDA_TRY(p, cudaMemsetAsync(p->d_range, 0, sizeof(u64), us));
                CUDA_TRY(p, cudaEventRecord(p->ev_upload, us));
            } else CUDA_TRY(p, cudaMemset(p->d_range, 0, sizeof(u64)));
        }
        p->dc.pconf = p->d_pconf;
        p->dc.n_pconf = np;
        CUDA_TRY(p, cudaEventCreateWithFlags(&p->ev_fork, cudaEventDisableTiming));
        CUDA_TRY(p, cudaEventCreateWithFlags(&p->ev_pre, cudaEventDisableTiming));
        CUDA_TRY(p, cudaEventCreateWithFlags(&p->ev_dec, cudaEventDisableTiming));
        for (size_t ci = 0; ci < p->classes.size(); ++ci) {
            auto &cl = p->classes[ci];
            cl.stream = pooled_stream(p->device, ci);
            if (!cl.stream) return fail(p, HAP_E_CUDA, "cudaStreamCreateWithFlags");
            CUDA_TRY(p, cudaEventCreateWithFlags(&cl.done, cudaEventDisableTiming));
        }
        if (tab_bytes) {
            // The prefix tree of a class depends on the cluster, the stage count, the model's layer kinds and the
            // window, not on the profiled tables: trees are kept per process under a key of exactly those inputs, so
            // that planning again on the same cluster (new tables, new batch) neither decodes the mappings for the
            // host nor rebuilds a tree.
            // the tree kernel holds times as doubles: exact while every prefix row stays below 2^52, which the
            // per-layer limit of 2^36 ns guarantees when N (2 + max tau) <= 2^16
            int tau_max = 0;
            for (int r = 0; r < p->prof.R; ++r) tau_max = std::max(tau_max, p->tau_q[r] >> 10);
            const bool rows_exact = (int64_t)N * (2 + tau_max) <= 65536;
            const bool want_trees = !(p->opts.flags & HAP_OPT_NO_TRIE) && p->dc.tau_linear && rows_exact;
            std::vector<TrieBuilt> built;
            std::vector<hap_problem::PpClass *> missing;
            std::vector<std::string> keys(p->classes.size());
            for (size_t ci = 0; ci < p->classes.size(); ++ci) {
                auto &cl = p->classes[ci];
                if (!cl.has_tab) continue;
                keys[ci] = trie_cache_key(p, cl);
                std::shared_ptr<const TrieClassHost> hit = trie_cache_find(keys[ci]);
                if (!hit) { missing.push_back(&cl); continue; }
                cl.masks_used = hit->masks_used;
                if (want_trees && !hit->parts.empty()) built.push_back(TrieBuilt{&cl, hit, class_plist(p, cl)});
            }
            if (!missing.empty()) {
                CUDA_TRY(p, uploads_done(p));                 // the decode below reads the configuration table
                for (const hap_problem::PpClass *cl : missing) {
                    const WorkItem &rep = p->items[cl->item_lo];
                    const u64 nmap = p->pconfs[rep.p].nmap;
                    maptab_kernel<<<(unsigned)((nmap + 3) / 4), 128>>>(p->dc, rep.p, nmap, p->d_maptab + cl->map_base);
                    CUDA_TRY(p, cudaGetLastError());
                    cl->tab_valid = true;
                }
                CUDA_TRY(p, cudaDeviceSynchronize());
                std::vector<uint8_t> tab(tab_bytes);
                CUDA_TRY(p, cudaMemcpy(tab.data(), p->d_maptab, tab_bytes, cudaMemcpyDeviceToHost));
                for (hap_problem::PpClass *clp : missing) {
                    auto &cl = *clp;
                    const u64 nmap = p->pconfs[p->items[cl.item_lo].p].nmap;
                    auto th = std::make_shared<TrieClassHost>();
                    // which type masks occur in a class: the DP kernel builds stage rows for those only
                    unsigned used = 0;
                    for (u64 e = 0; e < nmap * (u64)cl.PP; ++e) used |= 1u << tab[cl.map_base + e * 2];
                    th->masks_used = used;
                    cl.masks_used = used;
                    const std::vector<u32> plist = class_plist(p, cl);
                    const bool ok = want_trees && build_trie(p, cl, tab.data() + cl.map_base, nmap, plist.size(), *th);
                    if (!ok) th->parts.clear();
                    // a class whose tree was not wanted this time is not remembered as "has no tree"
                    if (want_trees) trie_cache_insert(keys[clp - p->classes.data()], th);
                    if (ok) built.push_back(TrieBuilt{&cl, th, plist});
                }
            }
            // the launch order of the merged decode / gather jobs follows the class order
            std::sort(built.begin(), built.end(), [](const TrieBuilt &x, const TrieBuilt &y) { return x.cl < y.cl; });
            std::string image_key = ekey;
            for (const auto &bc : built) image_key += keys[bc.cl - p->classes.data()];
            upload_tries(p, built, image_key);
        }
        p->n_pslots = 0;
        for (auto &cl : p->classes) {
            cl.pslot_lo = p->n_pslots;
            cl.pslot_n = cl.item_hi - cl.item_lo;
            if (cl.trie.ok) cl.pslot_n = std::max(cl.pslot_n, (size_t)cl.trie.n_conf * cl.trie.parts.size());
            p->n_pslots += cl.pslot_n;
        }
        if (p->n_pslots > p->n_partial) return fail(p, HAP_E_STATE, "partial-minimum slots exceed their allocation");
        p->enumerated = true;
    }
    if (n_pconf) *n_pconf = p->pconfs.size();
    if (n_candidates) *n_candidates = p->n_cand;
    return HAP_OK;
}

extern "C" hap_status hap_get_pconfs(const hap_problem *p, hap_pconf *host_out, uint64_t cap)
{
    if (!p || !host_out) return HAP_E_INVALID;
    if (!p->enumerated) return HAP_E_STATE;
    if (cap < p->pconfs.size()) return HAP_E_RANGE;
    std::memcpy(host_out, p->pconfs.data(), p->pconfs.size() * sizeof(hap_pconf));
    return HAP_OK;
}

static hap_status enter(hap_problem *p)
{
    if (!p) return HAP_E_INVALID;
    if (!p->enumerated) return fail(p, HAP_E_STATE, "hap_enumerate has not run");
    if (cudaSetDevice(p->device) != cudaSuccess) return fail(p, HAP_E_CUDA, "cudaSetDevice");
    if (uploads_done(p) != cudaSuccess) return fail(p, HAP_E_CUDA, "upload of the problem's tables");
    return HAP_OK;
}

static hap_status check_values(hap_problem *p)
{
    u64 flag = 0;
    CUDA_TRY(p, cudaMemcpy(&flag, p->d_range, sizeof(flag), cudaMemcpyDeviceToHost));
    if (flag) return fail(p, HAP_E_RANGE, "a layer time or stage coefficient exceeds the supported range (see hap.h)");
    return HAP_OK;
}

static hap_status check_range(hap_problem *p, uint64_t first, uint64_t count)
{
    if (first > p->n_cand || count > p->n_cand - first) return fail(p, HAP_E_RANGE, "candidate range outside [0, %llu)", (unsigned long long)p->n_cand);
    return HAP_OK;
}

extern "C" hap_status hap_decode(hap_problem *p, uint64_t first, uint64_t count, hap_candidate *dev_out, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return HAP_OK;
    if (!dev_out) return HAP_E_INVALID;
    const uint64_t blocks = (count + 3) / 4;
    if (blocks > 0x7fffffffull) return fail(p, HAP_E_RANGE, "count too large for one launch");
    decode_kernel<<<(unsigned)blocks, 128, 0, (cudaStream_t)stream>>>(p->dc, first, count, dev_out, nullptr);
    CUDA_TRY(p, cudaGetLastError());
    return HAP_OK;
}

// per (configuration, type) constants and stage coefficients, then the layer costs of `n_conf` configurations from
// `p_first` on (all by default); index_dev: of the one configuration that owns the candidate index stored there
static hap_status launch_layer_kernel(hap_problem *p, i64 *c2, double *c2f, bool quant, cudaStream_t st, i64 *lb_sum,
                                      const i64 *index_dev, unsigned p_first, unsigned n_conf, bool dependent)
{
    const unsigned thr = (unsigned)((p->model.N + 31) / 32 * 32);
    // programmatic dependent launch: the blocks start while type_const_kernel drains and wait inside the kernel
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(n_conf); cfg.blockDim = dim3(thr); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = dependent ? 1 : 0;
    const TypeConst *tcg = p->d_tc;
    i64 *no_i = nullptr; double *no_d = nullptr;
    // layer kinds: 0 all dense, 1 all MoE (uniform branch compiled away), 2 mixed
    const int kind = !p->dc.kind_uniform ? 2 : (p->kind[0] == HAP_MOE ? 1 : 0);
    using Fn = void (*)(const DevConst, const TypeConst *, i64 *, double *, i64 *, u64 *, const i64 *, unsigned);
    if (quant) {
        static const Fn fns[3][2] = {{layer_cost_kernel<true, 0, false>, layer_cost_kernel<true, 0, true>},
                                     {layer_cost_kernel<true, 1, false>, layer_cost_kernel<true, 1, true>},
                                     {layer_cost_kernel<true, 2, false>, layer_cost_kernel<true, 2, true>}};
        CUDA_TRY(p, cudaLaunchKernelEx(&cfg, fns[kind][lb_sum ? 1 : 0], p->dc, tcg, c2, no_d, lb_sum, p->d_range, index_dev, p_first));
    } else {
        static const Fn fns[3] = {layer_cost_kernel<false, 0, false>, layer_cost_kernel<false, 1, false>, layer_cost_kernel<false, 2, false>};
        CUDA_TRY(p, cudaLaunchKernelEx(&cfg, fns[kind], p->dc, tcg, no_i, c2f, no_i, p->d_range, index_dev, p_first));
    }
    return HAP_OK;
}

// configurations that own candidates of [first, first + count): a contiguous range [lo, hi)
static void configs_of_range(const hap_problem *p, u64 first, u64 count, unsigned &lo, unsigned &hi)
{
    auto owner = [&](u64 c) {
        size_t a = 0, b = p->pconfs.size();
        while (b - a > 1) { const size_t mid = (a + b) / 2; if (p->pconfs[mid].offset <= c) a = mid; else b = mid; }
        return (unsigned)a;
    };
    if (count == 0 || p->pconfs.empty()) { lo = hi = 0; return; }
    lo = owner(first); hi = owner(first + count - 1) + 1;
}

// Per-type constants and stage coefficients, then (where an output array is given) the layer costs, of the
// configurations [p_lo, p_hi): a pass over a candidate range touches only the configurations that own its candidates.
static hap_status launch_layer_costs(hap_problem *p, i64 *c2, i64 *coef, double *c2f, double *coeff, bool quant, cudaStream_t st,
                                     i64 *lb_sum = nullptr, unsigned p_lo = 0, unsigned p_hi = ~0u)
{
    if (p_hi > p->pconfs.size()) p_hi = (unsigned)p->pconfs.size();
    if (p_lo >= p_hi) return HAP_OK;
    const unsigned n_conf = p_hi - p_lo;
    const u64 nph = (u64)n_conf * HAP_MAX_TYPES;
    const unsigned b1 = (unsigned)((nph + kLcThreads - 1) / kLcThreads);
    if (quant) type_const_kernel<true><<<dim3(b1, 3), kLcThreads, 0, st>>>(p->dc, p->d_tc, coef, nullptr, p->d_range, p_lo, n_conf);
    else type_const_kernel<false><<<dim3(b1, 3), kLcThreads, 0, st>>>(p->dc, p->d_tc, nullptr, coeff, p->d_range, p_lo, n_conf);
    CUDA_TRY(p, cudaGetLastError());
    if ((quant && c2) || (!quant && c2f)) {
        hap_status s = launch_layer_kernel(p, c2, c2f, quant, st, lb_sum, nullptr, p_lo, n_conf, true);
        if (s != HAP_OK) return s;
    }
    CUDA_TRY(p, cudaGetLastError());
    return HAP_OK;
}

extern "C" hap_status hap_eval_layer_costs(hap_problem *p, int64_t *dev_c2, int64_t *dev_coef, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!dev_c2 && !dev_coef) return HAP_OK;
    return launch_layer_costs(p, (i64 *)dev_c2, (i64 *)dev_coef, nullptr, nullptr, true, (cudaStream_t)stream);
}

extern "C" hap_status hap_eval_layer_costs_f64(hap_problem *p, double *dev_c2, double *dev_coef, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!dev_c2 && !dev_coef) return HAP_OK;
    return launch_layer_costs(p, nullptr, nullptr, dev_c2, dev_coef, false, (cudaStream_t)stream);
}

// whether all candidates of the class lie outside the range the pass writes
static bool class_outside(const hap_problem *p, const hap_problem::PpClass &cl, const DpOut &out)
{
    const WorkItem &a = p->items[cl.item_lo], &b = p->items[cl.item_hi - 1];
    const u64 c0 = p->pconfs[a.p].offset, c1 = p->pconfs[b.p].offset + p->pconfs[b.p].nmap * (u64)p->opts.n_rc;
    return c1 <= out.first || c0 >= out.first + out.count;
}

// plain integer passes over more than one candidate walk the class's prefix tree; tables, refinement, fp64, cell
// counting and the one-candidate re-evaluation stay in pipeline_dp_kernel
static bool pass_uses_trie(const hap_problem *p, const hap_problem::PpClass &cl, const DpOut &out, bool f64)
{
    const bool refine = (p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT)) != 0 && !out.count_only && !out.force_plain;
    (void)f64;                                  // both value types walk the tree
    return cl.trie.ok && !out.count_only && !refine && p->dc.tau_linear != 0 && !out.dp_table && !out.choice && out.count > 1;
}

// Whether every class the pass touches walks its prefix tree: then the blocks of the tree kernel compute the layer
// times of their configuration themselves (Eq. 2 from the profiled tables and the per-type constants) and the pass
// neither writes nor reads the layer-cost array.
static bool pass_fuses_layer_costs(const hap_problem *p, const DpOut &out, bool search)
{
    if (p->opts.flags & HAP_OPT_NO_FUSE) return false;
    bool any = false;
    for (const auto &cl : p->classes) {
        if (!search && !out.first_dev && class_outside(p, cl, out)) continue;
        if (!pass_uses_trie(p, cl, out, false)) return false;
        any = true;
    }
    return any;
}

// candidate decode of a class for this pass, then its stage bytes into the class's tree
static hap_status launch_class_decode(hap_problem *p, const hap_problem::PpClass &cl)
{
    const hap_problem::Trie &tr = cl.trie;
    const uint8_t *tab = p->d_maptab + cl.map_base;
    const u64 nmap = p->pconfs[p->items[cl.item_lo].p].nmap;
    maptab_kernel<<<(unsigned)((nmap + 3) / 4), 128, 0, cl.stream>>>(p->dc, p->items[cl.item_lo].p, nmap, p->d_maptab + cl.map_base);
    CUDA_TRY(p, cudaGetLastError());
    for (const auto &pd : tr.parts) {
        const u32 n_g = pd.n_nodes + pd.n_cells + pd.nmap;
        TrieRowMap rmap;
        std::memcpy(rmap.mrow_of, pd.mrow_of, sizeof(rmap.mrow_of));
        trie_gather_kernel<<<(n_g + 255) / 256, 256, 0, cl.stream>>>(tab, cl.PP, pd.n_nodes, pd.n_cells, pd.nmap, pd.m_lo, pd.d_first_leaf,
                                                                      pd.d_depth, pd.d_gnode, rmap, pd.d_nodes, pd.d_cells, pd.d_leaves);
        CUDA_TRY(p, cudaGetLastError());
    }
    return HAP_OK;
}

// The candidate decode reads nothing the layer-cost kernels write: it waits only for the start of the pass (ev_pre,
// recorded before the layer-cost launches) and runs on the class streams beside the layer costs instead of between
// them and the recurrence.  On the host it is issued after the layer-cost launches, so that those reach an idle GPU
// without waiting for a dozen other launches to be queued.
static hap_status launch_decode_early(hap_problem *p, const DpOut &out, bool search)
{
    (void)search;
    bool any = false, all = true;
    for (const auto &cl : p->classes) {
        const bool uses = pass_uses_trie(p, cl, out, false);
        any |= uses;
        if (cl.trie.ok && !uses) all = false;
    }
    if (!any || !all || !p->n_gather_jobs || p->decode_jobs.n == 0) return HAP_OK;
    // one decode launch and one gather launch for all classes and parts, on the first class's stream
    cudaStream_t sx = p->classes[0].stream;
    CUDA_TRY(p, cudaStreamWaitEvent(sx, p->ev_pre, 0));
    const DecodeJobs &dj = p->decode_jobs;
    maptab_all_kernel<<<dj.blk_lo[dj.n], 128, 0, sx>>>(p->dc, dj, p->d_maptab);
    CUDA_TRY(p, cudaGetLastError());
    trie_gather_all_kernel<<<p->gather_blocks, 256, 0, sx>>>(p->d_gather_jobs, p->n_gather_jobs, p->d_maptab);
    CUDA_TRY(p, cudaGetLastError());
    CUDA_TRY(p, cudaEventRecord(p->ev_dec, sx));
    p->decoded_all = true;
    for (const auto &cl : p->classes) if (cl.trie.ok) cl.tab_valid = true;
    return HAP_OK;
}

// One launch per PP class (each has its own block shape); every block clips to the candidate range.
static hap_status launch_dp(hap_problem *p, const DpOut &out, bool search, cudaStream_t st, bool f64 = false)
{
    // the dynamic shared memory limit is a per-kernel, per-device attribute shared by every problem of the
    // process: raise it (never lower it) before a launch that needs more
    static size_t smem_limit[64][12];
    static std::mutex limit_mu;                 // both tables of raised limits, for problems used from several host threads
    std::lock_guard<std::mutex> limit_lock(limit_mu);
    const int dev = p->device & 63;
    // fork: every PP class runs on its own stream so that the tail of one class overlaps the next; a merged
    // candidate decode queued earlier in this pass joins first, so that the fork event covers it
    const bool decoded_all = p->decoded_all;
    p->decoded_all = false;
    if (decoded_all) CUDA_TRY(p, cudaStreamWaitEvent(st, p->ev_dec, 0));
    CUDA_TRY(p, cudaEventRecord(p->ev_fork, st));
    // the class with the most work goes first; the others fill the SMs it leaves free and its tail
    std::vector<const hap_problem::PpClass *> order;
    for (const auto &cl : p->classes) order.push_back(&cl);
    std::stable_sort(order.begin(), order.end(), [](const hap_problem::PpClass *a, const hap_problem::PpClass *b) {
        return (a->item_hi - a->item_lo) * (size_t)a->PP > (b->item_hi - b->item_lo) * (size_t)b->PP;
    });
    // a pruning search wants a good incumbent early: the lower bound S + (M-1) ceil(S / PP) falls with PP, so the
    // deepest pipelines are the likeliest to hold the best plan and go first
    if (search && out.prune)
        std::stable_sort(order.begin(), order.end(), [](const hap_problem::PpClass *a, const hap_problem::PpClass *b) { return a->PP > b->PP; });
    for (const hap_problem::PpClass *clp : order) {
        const hap_problem::PpClass &cl = *clp;
        // skip classes whose candidates all lie outside the range
        if (!search && !out.first_dev && class_outside(p, cl, out)) continue;     // (a range that starts at a device-side index: every class looks)
        const bool lin = p->dc.tau_linear != 0;
        const bool refine = (p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT)) != 0 && !out.count_only && !out.force_plain;
        const int variant = f64 ? 6 + (lin ? 1 : 0) : out.count_only ? 4 + (lin ? 1 : 0) : (refine ? 8 : 0) + (search ? 2 : 0) + (lin ? 1 : 0);
        const void *fn;
        if (f64) fn = lin ? (const void *)pipeline_dp_kernel<false, true, false, double> : (const void *)pipeline_dp_kernel<false, false, false, double>;
        else if (out.count_only) fn = lin ? (const void *)pipeline_dp_kernel<false, true, true> : (const void *)pipeline_dp_kernel<false, false, true>;
        else if (refine) fn = search ? (lin ? (const void *)pipeline_dp_kernel<true, true, false, i64, true> : (const void *)pipeline_dp_kernel<true, false, false, i64, true>)
                                     : (lin ? (const void *)pipeline_dp_kernel<false, true, false, i64, true> : (const void *)pipeline_dp_kernel<false, false, false, i64, true>);
        else fn = search ? (lin ? (const void *)pipeline_dp_kernel<true, true> : (const void *)pipeline_dp_kernel<true, false>)
                         : (lin ? (const void *)pipeline_dp_kernel<false, true> : (const void *)pipeline_dp_kernel<false, false>);
        if (cl.smem > smem_limit[dev][variant]) {
            CUDA_TRY(p, cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)cl.smem));
            smem_limit[dev][variant] = cl.smem;
        }
        const unsigned blocks = (unsigned)(cl.item_hi - cl.item_lo);
        const uint8_t *tab = cl.has_tab ? p->d_maptab + cl.map_base : nullptr;
        DpOut o = out;
        o.exact = (p->opts.flags & HAP_OPT_EXACT) != 0 && !out.force_plain;
        if (search) { o.partial_cost += cl.pslot_lo; o.partial_index += cl.pslot_lo; if (o.block_plan) o.block_plan += cl.pslot_lo; }
        if (pass_uses_trie(p, cl, out, f64)) {
            const hap_problem::Trie &tr = cl.trie;
            // 64 registers per thread in both shapes (measured: more warps per SM beat more registers per thread)
            const int tv = tr.threads > 512 ? 0 : 1;
            if (search && f64) return fail(p, HAP_E_STATE, "the fp64 search reduces a cost array");
            const bool counting = (p->opts.flags & HAP_OPT_COUNT_SPLITS) && !f64 && !search;
            const void *tfn = f64 ? (tv == 0 ? (const void *)trie_dp_kernel<false, 1024, 1, double> : (const void *)trie_dp_kernel<false, 512, 2, double>)
                            : search ? (tv == 0 ? (const void *)trie_dp_kernel<true, 1024, 1> : (const void *)trie_dp_kernel<true, 512, 2>)
                            : counting ? (tv == 0 ? (const void *)trie_dp_kernel<false, 1024, 1, i64, true> : (const void *)trie_dp_kernel<false, 512, 2, i64, true>)
                                       : (tv == 0 ? (const void *)trie_dp_kernel<false, 1024, 1> : (const void *)trie_dp_kernel<false, 512, 2>);
            static size_t trie_limit[64][8];
            const int vi = (f64 ? 4 : search ? 2 : counting ? 6 : 0) + tv;
            if (tr.smem > trie_limit[dev][vi]) {
                CUDA_TRY(p, cudaFuncSetAttribute(tfn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tr.smem));
                trie_limit[dev][vi] = tr.smem;
            }
            CUDA_TRY(p, cudaStreamWaitEvent(cl.stream, p->ev_fork, 0));
            if (!decoded_all) {                     // not queued beside the layer costs by this pass
                hap_status sd = launch_class_decode(p, cl);
                cl.tab_valid = true;
                if (sd != HAP_OK) return sd;
            }
            int n_parts = (int)tr.parts.size();
            unsigned n_active = tr.n_conf * (unsigned)n_parts;
            const u32 *plist = tr.d_plist;
            const TrieMeta *metas = tr.d_metas;
            void *c2v = f64 ? (void *)p->d_c2f : (void *)p->d_c2, *coefv = f64 ? (void *)p->d_coeff : (void *)p->d_coef;
            void *targs[] = {(void *)&p->dc, (void *)&plist, (void *)&n_active, (void *)&c2v, (void *)&p->d_coef, (void *)&coefv, (void *)&metas, (void *)&n_parts, (void *)&o};
            const unsigned tblocks = search ? (unsigned)cl.pslot_n : n_active;             // search: every partial slot of the class is written
            CUDA_TRY(p, cudaLaunchKernel(tfn, dim3(tblocks), dim3(tr.threads), targs, tr.smem, cl.stream));
            CUDA_TRY(p, cudaEventRecord(cl.done, cl.stream));
            CUDA_TRY(p, cudaStreamWaitEvent(st, cl.done, 0));
            continue;
        }
        const WorkItem *its = p->d_items + cl.item_lo;
        int nw = cl.warps;
        unsigned used = cl.masks_used;
        void *c2arg = f64 ? (void *)p->d_c2f : (void *)p->d_c2;
        void *cvarg = f64 ? (void *)p->d_coeff : (void *)p->d_coef;
        void *args[] = {(void *)&p->dc, (void *)&its, (void *)&c2arg, (void *)&p->d_coef, (void *)&cvarg, (void *)&tab, (void *)&o, (void *)&nw, (void *)&used};
        CUDA_TRY(p, cudaStreamWaitEvent(cl.stream, p->ev_fork, 0));
        if (cl.has_tab && (out.count > 1 || !cl.tab_valid)) {        // (a single candidate reuses a table that some pass has filled)
            // candidate decode (stage masks and link classes of every mapping of the class) is part of every pass,
            // not a cached result of hap_enumerate; the one-candidate re-evaluation of a winner reuses the table
            const WorkItem &rep = p->items[cl.item_lo];
            const u64 nmap = p->pconfs[rep.p].nmap;
            maptab_kernel<<<(unsigned)((nmap + 3) / 4), 128, 0, cl.stream>>>(p->dc, rep.p, nmap, p->d_maptab + cl.map_base);
            CUDA_TRY(p, cudaGetLastError());
            cl.tab_valid = true;
        }
        CUDA_TRY(p, cudaLaunchKernel(fn, dim3(blocks), dim3(cl.warps * 32), args, cl.smem, cl.stream));
        if (search && cl.pslot_n > blocks) {       // slots that only the class's tree kernel would write
            const unsigned extra = (unsigned)(cl.pslot_n - blocks);
            fill_partials_kernel<<<(extra + 255) / 256, 256, 0, cl.stream>>>(o.partial_cost + blocks, o.partial_index + blocks, extra);
            CUDA_TRY(p, cudaGetLastError());
        }
        CUDA_TRY(p, cudaEventRecord(cl.done, cl.stream));
        CUDA_TRY(p, cudaStreamWaitEvent(st, cl.done, 0));      // join
    }
    return HAP_OK;
}

extern "C" hap_status hap_pipeline_dp(hap_problem *p, uint64_t first, uint64_t count, int64_t *dev_cost,
                                      int64_t *dev_bottleneck, uint8_t *dev_partition, uint8_t *dev_recompute,
                                      int64_t *dev_dp_table, uint8_t *dev_choice, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return HAP_OK;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(p, cudaMemsetAsync(p->d_counters, 0, 8 * sizeof(u64), st));
    CUDA_TRY(p, cudaEventRecord(p->ev[0], st));
    DpOut out{};
    out.counters = p->d_counters;
    out.cost = (i64 *)dev_cost; out.bottleneck = (i64 *)dev_bottleneck; out.partition = dev_partition;
    out.recompute = dev_recompute; out.dp_table = (i64 *)dev_dp_table; out.choice = dev_choice;
    out.first = first; out.count = count;
    const bool fused = pass_fuses_layer_costs(p, out, false);
    out.tcg = fused ? p->d_tc : nullptr; out.range_flag = p->d_range;
    CUDA_TRY(p, cudaEventRecord(p->ev_pre, st));
    unsigned p_lo, p_hi;
    configs_of_range(p, first, count, p_lo, p_hi);
    if ((s = launch_layer_costs(p, fused ? nullptr : p->d_c2, p->d_coef, nullptr, nullptr, true, st, nullptr, p_lo, p_hi)) != HAP_OK) return s;
    CUDA_TRY(p, cudaEventRecord(p->ev[1], st));
    if ((s = launch_decode_early(p, out, false)) != HAP_OK) return s;
    if ((s = launch_dp(p, out, false, st)) != HAP_OK) return s;
    CUDA_TRY(p, cudaEventRecord(p->ev[2], st));
    p->timed = true;
    return HAP_OK;
}

static hap_status ensure_f64_buffers(hap_problem *p)
{
    const size_t np = p->pconfs.size();
    if (!p->d_c2f) CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_c2f, np * p->T * p->model.N * 2 * sizeof(double)));
    if (!p->d_coeff) CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_coeff, np * p->T * HAP_NCOEF * sizeof(double)));
    return HAP_OK;
}

extern "C" hap_status hap_pipeline_dp_f64(hap_problem *p, uint64_t first, uint64_t count, double *dev_cost,
                                          double *dev_bottleneck, uint8_t *dev_partition, uint8_t *dev_recompute,
                                          void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return HAP_OK;
    if (p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT)) return fail(p, HAP_E_INVALID, "the refinement passes exist in integer mode only");
    if ((s = ensure_f64_buffers(p)) != HAP_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(p, cudaMemsetAsync(p->d_counters, 0, 8 * sizeof(u64), st));
    CUDA_TRY(p, cudaEventRecord(p->ev[0], st));
    // the memory model stays on the integer byte coefficients; times stay unrounded
    DpOut out{};
    out.counters = p->d_counters;
    out.cost = (i64 *)dev_cost; out.bottleneck = (i64 *)dev_bottleneck; out.partition = dev_partition;
    out.recompute = dev_recompute; out.first = first; out.count = count;
    const bool fused = pass_fuses_layer_costs(p, out, false);
    out.tcg = fused ? p->d_tc : nullptr; out.range_flag = p->d_range;
    unsigned p_lo, p_hi;
    configs_of_range(p, first, count, p_lo, p_hi);
    if ((s = launch_layer_costs(p, nullptr, p->d_coef, nullptr, nullptr, true, st, nullptr, p_lo, p_hi)) != HAP_OK) return s;
    if ((s = launch_layer_costs(p, nullptr, nullptr, fused ? nullptr : p->d_c2f, p->d_coeff, false, st, nullptr, p_lo, p_hi)) != HAP_OK) return s;
    CUDA_TRY(p, cudaEventRecord(p->ev[1], st));
    if ((s = launch_dp(p, out, false, st, true)) != HAP_OK) return s;
    CUDA_TRY(p, cudaEventRecord(p->ev[2], st));
    p->timed = true;
    return HAP_OK;
}

extern "C" hap_status hap_search_range_f64(hap_problem *p, uint64_t first, uint64_t count, hap_plan *host_out,
                                           double *host_T_iter, double *host_bottleneck, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!host_out) return HAP_E_INVALID;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return fail(p, HAP_E_RANGE, "empty candidate range");
    cudaStream_t st = (cudaStream_t)stream;
    if (!p->d_fcost) CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_fcost, (size_t)p->n_cand * sizeof(i64)));
    if ((s = hap_pipeline_dp_f64(p, first, count, (double *)p->d_fcost, nullptr, nullptr, nullptr, stream)) != HAP_OK) return s;
    // non-negative doubles order like their bit patterns read as int64 (+inf is the largest), so the integer
    // (cost, index) argmin serves the fp64 costs unchanged
    if ((s = argmin_launch(p, p->d_fcost, count, p->d_best, st, 0x7fffffffffffffffll)) != HAP_OK) return s;
    i64 best[2];
    CUDA_TRY(p, cudaMemcpyAsync(best, p->d_best, sizeof(best), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(p, cudaStreamSynchronize(st));
    double bc;
    std::memcpy(&bc, &best[0], sizeof(bc));
    std::memset(host_out, 0, sizeof(*host_out));
    if (!(bc < 1.0e300)) return fail(p, HAP_E_INFEASIBLE, "no candidate satisfies the memory constraint");
    const u64 win = first + (u64)best[1];
    SingleOut *d1 = (SingleOut *)p->d_single;
    DpOut one{};
    one.cost = &d1->cost; one.bottleneck = &d1->bott; one.detail = d1->detail; one.partition = d1->part;
    one.recompute = d1->rec; one.first = win; one.count = 1;
    {   // the pass may have left the layer-cost array untouched: the winner's configuration is evaluated here
        size_t lo = 0, hi = p->pconfs.size();
        while (hi - lo > 1) { const size_t mid = (lo + hi) / 2; if (p->pconfs[mid].offset <= win) lo = mid; else hi = mid; }
        if ((s = launch_layer_kernel(p, nullptr, p->d_c2f, false, st, nullptr, nullptr, (unsigned)lo, 1, false)) != HAP_OK) return s;
    }
    if ((s = launch_dp(p, one, false, st, true)) != HAP_OK) return s;
    decode_kernel<<<1, 32, 0, st>>>(p->dc, win, 1, &d1->cand, nullptr);
    CUDA_TRY(p, cudaGetLastError());
    SingleOut h1;
    CUDA_TRY(p, cudaMemcpyAsync(&h1, d1, sizeof(h1), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(p, cudaStreamSynchronize(st));
    const hap_candidate &hc = h1.cand;
    const hap_pconf &pc = p->pconfs[hc.pconf];
    host_out->index = win;
    host_out->PP = pc.PP; host_out->TP = pc.TP; host_out->CP = pc.CP; host_out->DP = pc.DP; host_out->EP = pc.EP;
    host_out->TPE = pc.TPE; host_out->b = pc.b; host_out->M = pc.M; host_out->rc_mask = hc.rc_mask;
    std::memcpy(host_out->n, h1.part, HAP_MAX_PP);
    std::memcpy(host_out->r, h1.rec, HAP_MAX_PP);
    std::memcpy(host_out->mask, hc.mask, HAP_MAX_PP);
    double v[5];
    std::memcpy(&v[0], &h1.cost, 8); std::memcpy(&v[1], &h1.bott, 8); std::memcpy(&v[2], h1.detail, 24);
    host_out->T_iter = (int64_t)llrint(v[0]); host_out->bottleneck = (int64_t)llrint(v[1]);
    host_out->T_pipe = (int64_t)llrint(v[2]); host_out->T_sync = (int64_t)llrint(v[3]); host_out->T_opt = (int64_t)llrint(v[4]);
    if (host_T_iter) *host_T_iter = v[0];
    if (host_bottleneck) *host_bottleneck = v[1];
    return HAP_OK;
}

static hap_status joint_setup(hap_problem *p)
{
    if (p->joint_ready) return HAP_OK;
    const int T = p->T, N = p->model.N;
    size_t lmax_all = 0;
    std::vector<int> pps;
    for (const auto &r : p->pconfs) if (std::find(pps.begin(), pps.end(), r.PP) == pps.end()) pps.push_back(r.PP);
    for (int PP : pps) {
        const int64_t G = p->W / PP;
        bool homog = true;
        for (int h = 0; h < T; ++h) if (p->m[h] % G) homog = false;
        if (!homog) continue;
        hap_problem::JointHost jh;
        JointClass &jc = jh.jc;
        jc.PP = PP;
        int S = 1;
        for (int h = 0; h < HAP_MAX_TYPES; ++h) {
            jc.cnt[h] = h < T ? (int)(p->m[h] / G) : 0;
            jc.stride[h] = S;
            S *= jc.cnt[h] + 1;
            if (S > (1 << 22)) return fail(p, HAP_E_RANGE, "too many device states for the joint recurrence");
        }
        jc.S = S;
        std::vector<int> lvl_off(PP + 2, 0), st_idx(S), slot(S), level(S);
        for (int ui = 0; ui < S; ++ui) {
            int tot = 0;
            for (int h = 0; h < HAP_MAX_TYPES; ++h) tot += (ui / jc.stride[h]) % (jc.cnt[h] + 1);
            level[ui] = tot;
            lvl_off[tot + 1]++;
        }
        int lmax = 1;
        for (int l = 0; l <= PP; ++l) { lmax = std::max(lmax, lvl_off[l + 1]); lvl_off[l + 1] += lvl_off[l]; }
        std::vector<int> fill(lvl_off.begin(), lvl_off.end() - 1);
        for (int ui = 0; ui < S; ++ui) { slot[ui] = fill[level[ui]] - lvl_off[level[ui]]; st_idx[fill[level[ui]]++] = ui; }
        jc.lmax = lmax;
        lmax_all = std::max(lmax_all, (size_t)lmax);
        std::vector<int> arrays;
        arrays.insert(arrays.end(), lvl_off.begin(), lvl_off.end());
        arrays.insert(arrays.end(), st_idx.begin(), st_idx.end());
        arrays.insert(arrays.end(), slot.begin(), slot.end());
        for (int pos = 0; pos < S; ++pos) {                      // stage counts per type of the states, in level order
            int dg = 0;
            for (int h = 0; h < HAP_MAX_TYPES; ++h) dg |= ((st_idx[pos] / jc.stride[h]) % (jc.cnt[h] + 1)) << (8 * h);
            arrays.push_back(dg);
        }
        arrays.insert(arrays.end(), (size_t)S, 0);               // band table, filled by the kernel
        CUDA_TRY(p, cached_malloc(p->device, (void **)&jh.d_arrays, arrays.size() * sizeof(int)));
        CUDA_TRY(p, cudaMemcpy(jh.d_arrays, arrays.data(), arrays.size() * sizeof(int), cudaMemcpyHostToDevice));
        jc.lvl_off = jh.d_arrays; jc.st_idx = jh.d_arrays + (PP + 2); jc.slot = jc.st_idx + S;
        jc.dig = jc.slot + S; jc.band = jh.d_arrays + (PP + 2) + 3 * (size_t)S;
        for (size_t pi = 0; pi < p->pconfs.size(); ++pi) if (p->pconfs[pi].PP == PP) jh.ids.push_back((unsigned)pi);
        CUDA_TRY(p, cached_malloc(p->device, (void **)&jh.d_ids, jh.ids.size() * sizeof(unsigned)));
        CUDA_TRY(p, cudaMemcpy(jh.d_ids, jh.ids.data(), jh.ids.size() * sizeof(unsigned), cudaMemcpyHostToDevice));
        jh.smem = joint_smem_bytes(N, PP, T, p->prof.R, p->dc.tau_linear != 0);
        if (jh.smem > 227 * 1024) return fail(p, HAP_E_RANGE, "shared memory need of the joint recurrence exceeds the SM");
        p->joint.push_back(jh);
    }
    p->joint_grid = 2 * 148;
    if (lmax_all) {
        const size_t bytes = (size_t)p->joint_grid * 2 * lmax_all * T * (N + 1) * sizeof(i64);
        CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_joint_scratch, bytes));
    }
    p->joint_ready = true;
    return HAP_OK;
}

extern "C" hap_status hap_joint_bottleneck(hap_problem *p, int64_t *dev_out, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!dev_out) return HAP_E_INVALID;
    if ((s = joint_setup(p)) != HAP_OK) return s;
    cudaStream_t st = (cudaStream_t)stream;
    const size_t np = p->pconfs.size();
    CUDA_TRY(p, cudaMemsetAsync(dev_out, 0xff, np * p->opts.n_rc * sizeof(int64_t), st));     // -1: stages not homogeneous
    if ((s = launch_layer_costs(p, p->d_c2, p->d_coef, nullptr, nullptr, true, st)) != HAP_OK) return s;
    static size_t smem_limit[64][2];
    const int dev = p->device & 63;
    const bool lin = p->dc.tau_linear != 0;
    for (const auto &jh : p->joint) {
        const void *fn = lin ? (const void *)joint_dp_kernel<true> : (const void *)joint_dp_kernel<false>;
        if (jh.smem > smem_limit[dev][lin]) {
            CUDA_TRY(p, cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)jh.smem));
            smem_limit[dev][lin] = jh.smem;
        }
        const unsigned n_ids = (unsigned)jh.ids.size();
        const unsigned grid = std::min<unsigned>(n_ids, (unsigned)p->joint_grid);
        // scratch slices are sized for the widest class
        if (lin) joint_dp_kernel<true><<<grid, 256, jh.smem, st>>>(p->dc, jh.d_ids, n_ids, p->d_c2, p->d_coef, jh.jc, p->d_joint_scratch, (i64 *)dev_out);
        else joint_dp_kernel<false><<<grid, 256, jh.smem, st>>>(p->dc, jh.d_ids, n_ids, p->d_c2, p->d_coef, jh.jc, p->d_joint_scratch, (i64 *)dev_out);
        CUDA_TRY(p, cudaGetLastError());
    }
    return HAP_OK;
}

extern "C" hap_status hap_count_cells(hap_problem *p, uint64_t first, uint64_t count, uint64_t *host_cells, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!host_cells) return HAP_E_INVALID;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    *host_cells = 0;
    if (count == 0) return HAP_OK;
    cudaStream_t st = (cudaStream_t)stream;
    CUDA_TRY(p, cudaMemsetAsync(p->d_counters, 0, 8 * sizeof(u64), st));
    if ((s = launch_layer_costs(p, p->d_c2, p->d_coef, nullptr, nullptr, true, st)) != HAP_OK) return s;
    DpOut out{};
    out.counters = p->d_counters; out.first = first; out.count = count; out.count_only = 1;
    if ((s = launch_dp(p, out, false, st)) != HAP_OK) return s;
    CUDA_TRY(p, cudaMemcpyAsync(host_cells, p->d_counters + 4, sizeof(u64), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(p, cudaStreamSynchronize(st));
    return check_values(p);
}

extern "C" hap_status hap_get_timings(hap_problem *p, float *ms_layer_cost, float *ms_dp, uint64_t *cells)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!p->timed) return fail(p, HAP_E_STATE, "no hap_pipeline_dp or hap_search_* call to report on");
    CUDA_TRY(p, cudaEventSynchronize(p->ev[2]));
    if (ms_layer_cost) CUDA_TRY(p, cudaEventElapsedTime(ms_layer_cost, p->ev[0], p->ev[1]));
    if (ms_dp) CUDA_TRY(p, cudaEventElapsedTime(ms_dp, p->ev[1], p->ev[2]));
    if (cells) CUDA_TRY(p, cudaMemcpy(cells, p->d_counters + 4, sizeof(u64), cudaMemcpyDeviceToHost));
    return check_values(p);
}

extern "C" hap_status hap_eval_appendix_b(hap_problem *p, uint64_t first, uint64_t count, const uint8_t *dev_partition,
                                          const uint8_t *dev_recompute, int64_t *dev_t_iter, int64_t *dev_detail, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return HAP_OK;
    if (!dev_partition || !dev_recompute || !dev_t_iter) return HAP_E_INVALID;
    const uint64_t blocks = (count + 3) / 4;
    if (blocks > 0x7fffffffull) return fail(p, HAP_E_RANGE, "count too large for one launch");
    cudaStream_t st = (cudaStream_t)stream;
    if ((s = launch_layer_costs(p, p->d_c2, p->d_coef, nullptr, nullptr, true, st)) != HAP_OK) return s;
    appendix_b_kernel<<<(unsigned)blocks, 128, 0, st>>>(p->dc, first, count, p->d_c2, p->d_coef, dev_partition, dev_recompute,
                                                        (i64 *)dev_t_iter, (i64 *)dev_detail);
    CUDA_TRY(p, cudaGetLastError());
    return HAP_OK;
}

extern "C" hap_status hap_simulate_1f1b(hap_problem *p, uint64_t first, uint64_t count, const uint8_t *dev_partition,
                                        const uint8_t *dev_recompute, int64_t *dev_t_iter, int64_t *dev_detail, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return HAP_OK;
    if (!dev_partition || !dev_recompute || !dev_t_iter) return HAP_E_INVALID;
    if (count > 0x7fffffffull) return fail(p, HAP_E_RANGE, "count too large for one launch");
    cudaStream_t st = (cudaStream_t)stream;
    if ((s = launch_layer_costs(p, p->d_c2, p->d_coef, nullptr, nullptr, true, st)) != HAP_OK) return s;
    simulate_1f1b_kernel<<<(unsigned)count, 32, 0, st>>>(p->dc, first, count, p->d_c2, p->d_coef, dev_partition, dev_recompute,
                                                         (i64 *)dev_t_iter, (i64 *)dev_detail);
    CUDA_TRY(p, cudaGetLastError());
    return HAP_OK;
}

// ------------------------------------------------------------------------------------------
// hap_problem_save / hap_problem_load: the planner's inputs as one flat blob (the profiled tables are the
// expensive part of a planning problem: Sec. 4 caches them between runs)
// ------------------------------------------------------------------------------------------
namespace {
constexpr uint64_t kBlobMagic = 0x31424f4c42504148ull;        // "HAPBLOB1"
struct BlobWriter {
    unsigned char *buf; uint64_t cap, at = 0;
    void bytes(const void *src, uint64_t n) { if (buf && at + n <= cap) std::memcpy(buf + at, src, n); at += n; }
    template <class T> void pod(const T &v) { bytes(&v, sizeof(T)); }
    template <class T> void vec(const std::vector<T> &v) { pod<uint64_t>(v.size()); if (!v.empty()) bytes(v.data(), v.size() * sizeof(T)); }
};
struct BlobReader {
    const unsigned char *buf; uint64_t len, at = 0; bool ok = true;
    void bytes(void *dst, uint64_t n) { if (!ok || n > len - at) { ok = false; return; } std::memcpy(dst, buf + at, n); at += n; }
    template <class T> void pod(T &v) { bytes(&v, sizeof(T)); }
    template <class T> void vec(std::vector<T> &v, uint64_t max_n)
    {
        uint64_t n = 0; pod(n);
        if (!ok || n > max_n || n * sizeof(T) > len - at) { ok = false; return; }
        v.resize(n);
        if (n) bytes(v.data(), n * sizeof(T));
    }
};
}  // namespace

extern "C" hap_status hap_problem_save(hap_problem *p, void *host_buf, uint64_t cap, uint64_t *host_need)
{
    if (!p || !host_need) return HAP_E_INVALID;
    if (cudaSetDevice(p->device) != cudaSuccess) return fail(p, HAP_E_CUDA, "cudaSetDevice");
    const int N = p->model.N, T = p->T;
    const hap_profile &pf = p->prof;
    const size_t n4 = (size_t)T * pf.ntp * pf.ncp * pf.nmb, n5 = n4 * N;
    // the tables live on the device only (per-layer ones interleaved entry by entry): read them back in the caller's layout
    std::vector<double> dev(4 * n5 + 2 * n4), tab[4];
    CUDA_TRY(p, uploads_done(p));
    CUDA_TRY(p, cudaMemcpy(dev.data(), p->d_tables, dev.size() * sizeof(double), cudaMemcpyDeviceToHost));
    for (int t = 0; t < 4; ++t) { tab[t].resize(n5); for (size_t i = 0; i < n5; ++i) tab[t][i] = dev[4 * i + t]; }
    std::vector<double> tpre(dev.begin() + 4 * n5, dev.begin() + 4 * n5 + n4), tpost(dev.begin() + 4 * n5 + n4, dev.end());
    std::vector<double> fsize(p->dc.fsize, p->dc.fsize + pf.n_fsize), feff;
    for (int c = 0; c < 3; ++c) feff.insert(feff.end(), p->dc.feff[c], p->dc.feff[c] + pf.n_fsize);
    BlobWriter w{static_cast<unsigned char *>(host_buf), host_buf ? cap : 0};
    w.pod(kBlobMagic); w.pod<uint64_t>(0);                         // total size, patched below
    hap_model mo = p->model; mo.kind = nullptr;
    w.pod(mo); w.vec(p->kind);
    w.pod<int32_t>(T);
    w.vec(p->P); w.vec(p->C); w.vec(p->node_size); w.vec(p->bw_intra); w.vec(p->node_type); w.vec(p->node_bw_inter);
    w.vec(p->tp_list); w.vec(p->cp_list); w.vec(p->mb_list); w.vec(p->ep_list);
    for (int t = 0; t < 4; ++t) w.vec(tab[t]);
    w.vec(tpre); w.vec(tpost);
    w.vec(p->eta); w.vec(p->croute); w.vec(p->alpha); w.vec(p->rho); w.vec(p->act_coef); w.vec(p->copt); w.vec(p->cap_eff);
    w.vec(p->xi_q); w.vec(p->tau_q); w.vec(fsize); w.vec(feff);
    const double scal[7] = {pf.kappa, pf.chi, pf.gamma, pf.ovl_tp, pf.ovl_cp, pf.ovl_dp, pf.capf};
    w.bytes(scal, sizeof(scal));
    w.vec(p->pp_list); w.vec(p->tpe_list); w.vec(p->rc_masks);
    const hap_search_opts &so = p->opts;
    const int64_t oi[6] = {so.tp_max, so.delta_q, (int64_t)so.map_cap, so.prune, so.flags, so.eta_q};
    w.bytes(oi, sizeof(oi));
    *host_need = w.at;
    if (!host_buf || cap < w.at) return host_buf ? fail(p, HAP_E_RANGE, "the blob needs %llu bytes", (unsigned long long)w.at) : HAP_OK;
    std::memcpy(static_cast<unsigned char *>(host_buf) + 8, &w.at, 8);
    return HAP_OK;
}

extern "C" hap_status hap_problem_load(const void *host_buf, uint64_t len, hap_problem **out)
{
    if (!out) return HAP_E_INVALID;
    *out = nullptr;
    if (!host_buf || len < 16) return HAP_E_INVALID;
    BlobReader r{static_cast<const unsigned char *>(host_buf), len};
    uint64_t magic = 0, total = 0;
    r.pod(magic); r.pod(total);
    if (!r.ok || magic != kBlobMagic || total != len) return HAP_E_INVALID;
    constexpr uint64_t kMaxTab = 1ull << 28;
    hap_model mo{}; std::vector<uint8_t> kind;
    int32_t T = 0;
    std::vector<int64_t> P, C, cap_eff;
    std::vector<int32_t> node_size, node_type, tp, cp, mb, ep, xi, tau, pp, tpe;
    std::vector<double> bw_intra, node_bw, tab[4], tpre, tpost, eta, croute, alpha, rho, act, copt, fsize, feff;
    std::vector<uint32_t> rc;
    r.pod(mo); r.vec(kind, HAP_MAX_LAYERS);
    r.pod(T);
    r.vec(P, HAP_MAX_TYPES); r.vec(C, HAP_MAX_TYPES); r.vec(node_size, HAP_MAX_TYPES); r.vec(bw_intra, HAP_MAX_TYPES);
    r.vec(node_type, 1u << 20); r.vec(node_bw, 1u << 20);
    r.vec(tp, HAP_MAX_LIST); r.vec(cp, HAP_MAX_LIST); r.vec(mb, HAP_MAX_LIST); r.vec(ep, HAP_MAX_LIST);
    for (int t = 0; t < 4; ++t) r.vec(tab[t], kMaxTab);
    r.vec(tpre, kMaxTab); r.vec(tpost, kMaxTab);
    r.vec(eta, HAP_MAX_TYPES); r.vec(croute, HAP_MAX_TYPES); r.vec(alpha, 3); r.vec(rho, HAP_MAX_LIST); r.vec(act, 2);
    r.vec(copt, HAP_MAX_TYPES); r.vec(cap_eff, HAP_MAX_TYPES);
    r.vec(xi, HAP_MAX_RC); r.vec(tau, HAP_MAX_RC); r.vec(fsize, HAP_MAX_LIST); r.vec(feff, 3 * HAP_MAX_LIST);
    double scal[7] = {0}; r.bytes(scal, sizeof(scal));
    r.vec(pp, HAP_MAX_LIST); r.vec(tpe, HAP_MAX_LIST); r.vec(rc, HAP_MAX_RC_MASKS);
    int64_t oi[6] = {0}; r.bytes(oi, sizeof(oi));
    if (!r.ok || r.at != len) return HAP_E_INVALID;
    // sizes that hap_problem_create takes on trust from the pointers it is given
    if (T < 1 || T > HAP_MAX_TYPES || mo.N < 1 || (int64_t)kind.size() != mo.N || (int)P.size() != T || (int)C.size() != T ||
        (int)node_size.size() != T || (int)bw_intra.size() != T || node_type.size() != node_bw.size() || (int)eta.size() != T ||
        (int)croute.size() != T || alpha.size() != 3 || rho.size() != ep.size() || act.size() != 2 || (int)copt.size() != T ||
        (int)cap_eff.size() != T || xi.size() != tau.size() || xi.empty() || feff.size() != 3 * fsize.size())
        return HAP_E_INVALID;
    const size_t n4 = (size_t)T * tp.size() * cp.size() * mb.size(), n5 = n4 * (size_t)mo.N;
    for (int t = 0; t < 4; ++t) if (tab[t].size() != n5) return HAP_E_INVALID;
    if (tpre.size() != n4 || tpost.size() != n4) return HAP_E_INVALID;
    mo.kind = kind.data();
    hap_cluster cl{};
    cl.n_types = T; cl.P = P.data(); cl.C = C.data(); cl.node_size = node_size.data(); cl.bw_intra = bw_intra.data();
    cl.n_nodes = (int32_t)node_type.size(); cl.node_type = node_type.data(); cl.node_bw_inter = node_bw.data();
    hap_profile pf{};
    pf.ntp = (int32_t)tp.size(); pf.ncp = (int32_t)cp.size(); pf.nmb = (int32_t)mb.size(); pf.nep = (int32_t)ep.size();
    pf.tp_list = tp.data(); pf.cp_list = cp.data(); pf.mb_list = mb.data(); pf.ep_list = ep.data();
    pf.tdf = tab[0].data(); pf.tdb = tab[1].data(); pf.tff = tab[2].data(); pf.tfb = tab[3].data();
    pf.tpre = tpre.data(); pf.tpost = tpost.data();
    pf.eta = eta.data(); pf.croute = croute.data(); pf.kappa = scal[0]; pf.alpha = alpha.data(); pf.chi = scal[1];
    pf.rho = rho.data(); pf.gamma = scal[2]; pf.ovl_tp = scal[3]; pf.ovl_cp = scal[4]; pf.ovl_dp = scal[5];
    pf.act_coef = act.data(); pf.capf = scal[6]; pf.copt = copt.data(); pf.cap_eff = cap_eff.data();
    pf.R = (int32_t)xi.size(); pf.xi_q = xi.data(); pf.tau_q = tau.data();
    pf.n_fsize = (int32_t)fsize.size(); pf.fsize = fsize.empty() ? nullptr : fsize.data(); pf.feff = feff.empty() ? nullptr : feff.data();
    hap_search_opts so{};
    so.npp = (int32_t)pp.size(); so.ntpe = (int32_t)tpe.size(); so.pp_list = pp.data(); so.tpe_list = tpe.data();
    so.tp_max = (int32_t)oi[0]; so.delta_q = (int32_t)oi[1]; so.map_cap = (uint64_t)oi[2]; so.n_rc = (int32_t)rc.size();
    so.rc_masks = rc.data(); so.prune = (int32_t)oi[3]; so.flags = (int32_t)oi[4]; so.eta_q = (int32_t)oi[5];
    return hap_problem_create(&mo, &cl, &pf, &so, out);
}

extern "C" hap_status hap_problem_dims(const hap_problem *p, int32_t *host_N, int32_t *host_T, int32_t *host_n_rc)
{
    if (!p) return HAP_E_INVALID;
    if (host_N) *host_N = p->model.N;
    if (host_T) *host_T = p->T;
    if (host_n_rc) *host_n_rc = p->opts.n_rc;
    return HAP_OK;
}

extern "C" hap_status hap_self_check(uint64_t *host_sites)
{
    if (!host_sites) return HAP_E_INVALID;
    *host_sites = 0;
#ifdef HAP_CHECKED
    if (cudaDeviceSynchronize() != cudaSuccess) return HAP_E_CUDA;
    unsigned long long sites = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&sites, hap::g_hap_check_sites, sizeof(sites)) != cudaSuccess) return HAP_E_CUDA;
    if (cudaMemcpyToSymbol(hap::g_hap_check_sites, &zero, sizeof(zero)) != cudaSuccess) return HAP_E_CUDA;
    *host_sites = sites;
    return HAP_OK;
#else
    return HAP_E_STATE;                     // the checks are compiled away in this build
#endif
}

extern "C" hap_status hap_launches_per_pass(hap_problem *p, uint32_t *host_count)
{
    if (!p || !host_count) return HAP_E_INVALID;
    if (!p->enumerated) return fail(p, HAP_E_STATE, "hap_enumerate has not run");
    const bool lin = p->dc.tau_linear != 0;
    const bool refine = (p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT)) != 0;
    uint32_t n = 2 + 2;                                     // type constants, layer costs; argmin partial and final
    bool all_trees = p->n_gather_jobs > 0;
    for (const auto &cl : p->classes) if (cl.trie.ok && !(lin && !refine)) all_trees = false;
    bool fused = !(p->opts.flags & HAP_OPT_NO_FUSE) && lin && !refine && !p->classes.empty();
    for (const auto &cl : p->classes) if (!cl.trie.ok) fused = false;
    if (fused) n -= 1;                                      // the tree blocks compute the layer costs themselves
    if (all_trees) n += 2;                                  // one decode and one tree-gather launch for all classes
    for (const auto &cl : p->classes) {
        if (cl.trie.ok && lin && !refine) n += all_trees ? 1 : 1 + (uint32_t)cl.trie.parts.size() + 1;   // (decode, gather per part,) tree DP
        else n += (cl.has_tab ? 1 : 0) + 1;                                            // decode table, one-warp-per-candidate DP
    }
    *host_count = n;
    return HAP_OK;
}

static hap_status argmin_launch(hap_problem *p, const i64 *dev_cost, uint64_t count, i64 *dev_out, cudaStream_t st, i64 init)
{
    const unsigned blocks = (unsigned)std::min<uint64_t>((count + 255) / 256, 1024);
    argmin_partial_kernel<<<blocks, 256, 0, st>>>(dev_cost, count, p->d_pcost, p->d_pindex, init);
    CUDA_TRY(p, cudaGetLastError());
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(1); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    const i64 *pc = p->d_pcost; const u64 *pi = p->d_pindex; const u64 nb = blocks;
    const PlanSlot *no_plans = nullptr; i64 *no_vals = nullptr; uint8_t *no_bytes = nullptr;
    CUDA_TRY(p, cudaLaunchKernelEx(&cfg, argmin_final_kernel, pc, pi, nb, dev_out, init, no_plans, no_vals, no_bytes, no_bytes));
    return HAP_OK;
}

extern "C" hap_status hap_argmin(hap_problem *p, const int64_t *dev_cost, uint64_t count, int64_t *dev_out, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!dev_cost || !dev_out || count == 0) return HAP_E_INVALID;
    return argmin_launch(p, (const i64 *)dev_cost, count, (i64 *)dev_out, (cudaStream_t)stream, kInf);
}

extern "C" hap_status hap_search_range(hap_problem *p, uint64_t first, uint64_t count, hap_plan *host_out,
                                       hap_search_stats *host_stats, void *stream)
{
    hap_status s = enter(p);
    if (s != HAP_OK) return s;
    if (!host_out) return HAP_E_INVALID;
    if ((s = check_range(p, first, count)) != HAP_OK) return s;
    if (count == 0) return fail(p, HAP_E_RANGE, "empty candidate range");
    cudaStream_t st = (cudaStream_t)stream;
    std::memset(host_out, 0, sizeof(*host_out));
    const u64 init_counters[8] = {0, 0, 0, (u64)kInf, 0, 0, 0, 0};           // [3] = incumbent starts at +INF
    CUDA_TRY(p, cudaMemcpyAsync(p->d_counters, init_counters, sizeof(init_counters), cudaMemcpyHostToDevice, st));
    CUDA_TRY(p, cudaEventRecord(p->ev[0], st));
    DpOut out{};
    out.lb_sum = p->d_lb;
    out.first = first; out.count = count; out.prune = p->opts.prune;
    out.partial_cost = p->d_pcost; out.partial_index = p->d_pindex; out.counters = p->d_counters;
    out.incumbent = p->d_counters + 3;
    const bool refine_mode = (p->opts.flags & (HAP_OPT_REFINE | HAP_OPT_EXACT)) != 0;
    const bool fused = pass_fuses_layer_costs(p, out, true);
    out.tcg = fused ? p->d_tc : nullptr; out.range_flag = p->d_range;
    CUDA_TRY(p, cudaEventRecord(p->ev_pre, st));
    unsigned p_lo, p_hi;
    configs_of_range(p, first, count, p_lo, p_hi);
    if (refine_mode && count > 1) { p_lo = 0; p_hi = ~0u; }          // (the bounds kernel below reads every configuration's S)
    if ((s = launch_layer_costs(p, fused ? nullptr : p->d_c2, p->d_coef, nullptr, nullptr, true, st, fused ? nullptr : p->d_lb, p_lo, p_hi)) != HAP_OK) return s;
    CUDA_TRY(p, cudaEventRecord(p->ev[1], st));
    if (refine_mode && count > 1) {
        // The refinement and the exact sweep cost one warp per candidate and up to dozens of passes each, so they run
        // only where they can matter.  A plain pass over the prefix trees leaves every candidate's bottleneck B*; with
        // S the configuration's lower bound on the stage-cost sum, no partition of the candidate gets below
        // S + (M-1) B* (sync and optimizer terms only add).  The candidate with the smallest bound is evaluated first
        // and its cost starts the incumbent; the refinement kernels then skip every candidate whose bound exceeds the
        // incumbent (strict, so the (cost, index) minimum is unchanged).
        if (!p->d_cand_lb) CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_cand_lb, (size_t)p->n_cand * sizeof(i64)));
        DpOut plain{};
        plain.bottleneck = p->d_cand_lb + first;         // the kernels index outputs by candidate - first: entry c of the array
        plain.first = first; plain.count = count; plain.force_plain = 1; plain.range_flag = p->d_range;
        if ((s = launch_decode_early(p, plain, false)) != HAP_OK) return s;
        if ((s = launch_dp(p, plain, false, st)) != HAP_OK) return s;
        cand_bound_kernel<<<(unsigned)p->pconfs.size(), 128, 0, st>>>(p->dc, p->d_lb, p->d_cand_lb, first, count);
        CUDA_TRY(p, cudaGetLastError());
        if ((s = argmin_launch(p, p->d_cand_lb + first, count, p->d_best, st, kInf)) != HAP_OK) return s;
        offset_index_kernel<<<1, 32, 0, st>>>(p->d_best + 1, (i64)first);
        SingleOut *d0 = (SingleOut *)p->d_single;
        DpOut seed{};
        seed.cost = &d0->cost; seed.first = 0; seed.count = 1; seed.first_dev = p->d_best + 1;
        if ((s = launch_dp(p, seed, false, st)) != HAP_OK) return s;
        set_incumbent_kernel<<<1, 32, 0, st>>>(p->d_counters + 3, &d0->cost, p->d_best + 1);
        CUDA_TRY(p, cudaGetLastError());
        out.cand_lb = p->d_cand_lb;
    }
    // When every class of the search walks its prefix tree, each block also leaves the plan of its best candidate
    // (partition, levels, the terms of Eq. 4) and the final reduction copies the winner's: nothing is evaluated twice.
    bool plans = count > 1;
    for (const auto &cl : p->classes) plans = plans && pass_uses_trie(p, cl, out, false);
    SingleOut *d1 = (SingleOut *)p->d_single;
    if (plans) {
        if (!p->d_plans) CUDA_TRY(p, cached_malloc(p->device, (void **)&p->d_plans, p->n_pslots * sizeof(PlanSlot)));
        out.block_plan = p->d_plans;
    }
    if ((s = launch_decode_early(p, out, true)) != HAP_OK) return s;
    if ((s = launch_dp(p, out, true, st)) != HAP_OK) return s;
    static_assert(offsetof(SingleOut, bott) == 8 && offsetof(SingleOut, detail) == 16, "the final reduction writes cost, bottleneck and the three terms in a row");
    if (plans) argmin_final_kernel<<<1, 256, 0, st>>>(p->d_pcost, p->d_pindex, p->n_pslots, p->d_best, kInf, p->d_plans, &d1->cost, d1->part, d1->rec);
    else argmin_final_kernel<<<1, 256, 0, st>>>(p->d_pcost, p->d_pindex, p->n_pslots, p->d_best, kInf);
    CUDA_TRY(p, cudaGetLastError());
    CUDA_TRY(p, cudaEventRecord(p->ev[2], st));
    p->timed = true;
    if (!plans) {
        // the winner is evaluated once more alone, for its partition and recomputation levels; its index stays on the
        // device (every class's kernel looks whether the index is its own), so the host waits only once
        DpOut one{};
        one.cost = &d1->cost; one.bottleneck = &d1->bott; one.detail = d1->detail; one.partition = d1->part;
        one.recompute = d1->rec; one.first = 0; one.count = 1; one.first_dev = p->d_best + 1;
        if (fused && (s = launch_layer_kernel(p, p->d_c2, nullptr, true, st, nullptr, p->d_best + 1, 0, 1, false)) != HAP_OK) return s;
        if ((s = launch_dp(p, one, false, st)) != HAP_OK) return s;
    }
    decode_kernel<<<1, 32, 0, st>>>(p->dc, 0, 1, &d1->cand, p->d_best + 1);
    CUDA_TRY(p, cudaGetLastError());
    // range flag, counters, minimum and the re-evaluated winner sit in consecutive 256-byte slots at the end of the
    // arena: one copy brings all four back
    alignas(16) unsigned char tail[3 * 256 + sizeof(SingleOut)];
    if ((unsigned char *)p->d_counters - (unsigned char *)p->d_range != 256 || (unsigned char *)p->d_best - (unsigned char *)p->d_range != 512 ||
        (unsigned char *)p->d_single - (unsigned char *)p->d_range != 768)
        return fail(p, HAP_E_STATE, "result slots are not adjacent");
    CUDA_TRY(p, cudaMemcpyAsync(tail, p->d_range, sizeof(tail), cudaMemcpyDeviceToHost, st));
    CUDA_TRY(p, cudaStreamSynchronize(st));
    i64 best[2];
    u64 counters[4], flag = 0;
    SingleOut h1;
    std::memcpy(&flag, tail, sizeof(flag));
    std::memcpy(counters, tail + 256, sizeof(counters));
    std::memcpy(best, tail + 512, sizeof(best));
    std::memcpy(&h1, tail + 768, sizeof(h1));
    if (host_stats) {
        std::memset(host_stats, 0, sizeof(*host_stats));
        host_stats->n_pconf = p->pconfs.size(); host_stats->n_candidates = p->n_cand;
        host_stats->n_evaluated = counters[0]; host_stats->n_feasible = counters[1]; host_stats->n_pruned = counters[2];
        cudaEventElapsedTime(&host_stats->ms_layer_cost, p->ev[0], p->ev[1]);
        cudaEventElapsedTime(&host_stats->ms_dp, p->ev[1], p->ev[2]);
        host_stats->ms_total = host_stats->ms_layer_cost + host_stats->ms_dp;
    }
    if (flag) return fail(p, HAP_E_RANGE, "a layer time or stage coefficient exceeds the supported range (see hap.h)");
    if (best[0] >= kInf) return fail(p, HAP_E_INFEASIBLE, "no candidate satisfies the memory constraint");
    const u64 win = (u64)best[1];
    const hap_candidate &hc = h1.cand;
    if (h1.cost != best[0] || hc.index != win) return fail(p, HAP_E_CUDA, "winner re-evaluation disagrees with the search");
    const hap_pconf &pc = p->pconfs[hc.pconf];
    host_out->index = win;
    host_out->PP = pc.PP; host_out->TP = pc.TP; host_out->CP = pc.CP; host_out->DP = pc.DP; host_out->EP = pc.EP;
    host_out->TPE = pc.TPE; host_out->b = pc.b; host_out->M = pc.M; host_out->rc_mask = hc.rc_mask;
    std::memcpy(host_out->n, h1.part, HAP_MAX_PP);
    std::memcpy(host_out->r, h1.rec, HAP_MAX_PP);
    std::memcpy(host_out->mask, hc.mask, HAP_MAX_PP);
    host_out->T_iter = h1.cost; host_out->bottleneck = h1.bott;
    host_out->T_pipe = h1.detail[0]; host_out->T_sync = h1.detail[1]; host_out->T_opt = h1.detail[2];
    return HAP_OK;
}

extern "C" hap_status hap_search_best(hap_problem *p, hap_plan *host_out, hap_search_stats *host_stats, void *stream)
{
    if (!p) return HAP_E_INVALID;
    if (!p->enumerated) return fail(p, HAP_E_STATE, "hap_enumerate has not run");
    return hap_search_range(p, 0, p->n_cand, host_out, host_stats, stream);
}

// ------------------------------------------------------------------------------------------
// hap_argmin_static: the (cost, index) minimum without any allocation
// ------------------------------------------------------------------------------------------
// Scratch for the per-block partial minima lives in the library image itself.  Every device that
// loads the library carries these 64 KiB until the process exits.
constexpr unsigned kStaticArgminTile = 16384;                                   // costs per block
constexpr unsigned kStaticArgminBlocks = (unsigned)(HAP_ARGMIN_STATIC_MAX_COUNT / kStaticArgminTile);
static __device__ __align__(256) unsigned char g_argmin_static_scratch[kStaticArgminBlocks * 16];

// In host code the name above is only a handle for the runtime, not an address a kernel can use.
// The device address is looked up once per device (with that device current) and cached here.
// The entry point has no handle, so it is the one most likely to be called from several host threads: the lookup
// is serialised (a lock per call costs nothing beside two kernel launches).
static void *g_argmin_static_ptr[64];
static bool g_argmin_static_ready[64];
static std::mutex g_argmin_static_mu;

extern "C" hap_status hap_argmin_static(const int64_t *dev_cost, uint64_t count, int64_t *dev_out, void *stream)
{
    if (!dev_cost || !dev_out) return HAP_E_INVALID;
    if (count == 0 || count > HAP_ARGMIN_STATIC_MAX_COUNT) return HAP_E_RANGE;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return HAP_E_CUDA;
    if (dev < 0 || dev >= 64) return HAP_E_RANGE;
    void *scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_argmin_static_mu);
        if (!g_argmin_static_ready[dev]) {
            void *ptr = nullptr;
            if (cudaGetSymbolAddress(&ptr, g_argmin_static_scratch) != cudaSuccess || !ptr) return HAP_E_CUDA;
            g_argmin_static_ptr[dev] = ptr;
            g_argmin_static_ready[dev] = true;
        }
        scratch = g_argmin_static_ptr[dev];
    }
    {   // the cost array must live on the current device (the scratch and the launches do)
        cudaPointerAttributes at{};
        if (cudaPointerGetAttributes(&at, dev_cost) != cudaSuccess) { cudaGetLastError(); return HAP_E_INVALID; }
        if (at.type == cudaMemoryTypeDevice && at.device != dev) return HAP_E_INVALID;
    }
    i64 *pcost = reinterpret_cast<i64 *>(scratch);
    u64 *pindex = reinterpret_cast<u64 *>(pcost + kStaticArgminBlocks);
    cudaStream_t st = (cudaStream_t)stream;
    const unsigned blocks = (unsigned)((count + kStaticArgminTile - 1) / kStaticArgminTile);
    // every partial that the second kernel reads is written by the first one in this same call, so
    // nothing left in the scratch by an earlier call is ever read and nothing has to be cleared
    argmin_partial_kernel<<<blocks, 256, 0, st>>>((const i64 *)dev_cost, count, pcost, pindex, kInf);
    if (cudaGetLastError() != cudaSuccess) return HAP_E_CUDA;
    argmin_final_kernel<<<1, 256, 0, st>>>(pcost, pindex, blocks, (i64 *)dev_out, kInf);
    if (cudaGetLastError() != cudaSuccess) return HAP_E_CUDA;
    return HAP_OK;
}

// Host side of the C ABI declared in include/bns.h: argument validation, launch planning, workspace
// layout and kernel launches.  Nothing here allocates device memory or synchronises the host (except
// the two calls that are documented to: bns_workspace_status and bns_profile_read).
#include "bns.h"

#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>
#include <vector>

#include "bns_kernels.cuh"
#include "bns_nhwc_kernels.cuh"
#include "bns_slab_kernels.cuh"

namespace {

using namespace bns;

constexpr size_t kAlign = 256;
constexpr size_t kHeaderBytes = 256;  // status word lives at the start of the workspace
constexpr int kMaxDevices = 64;
constexpr int kSmCountFallback = 148;     // B200; used only if the device cannot be queried

// Streaming multiprocessors of the current device (queried once per device).
int sm_count() {
    static std::atomic<int> cached[kMaxDevices];
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) return kSmCountFallback;
    int n = cached[device].load(std::memory_order_relaxed);
    if (n > 0) return n;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, device) != cudaSuccess || n <= 0) {
        cudaGetLastError();
        return kSmCountFallback;
    }
    cached[device].store(n, std::memory_order_relaxed);
    return n;
}

size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
int elem_bytes(int dtype) { return dtype == BNS_F32 ? 4 : 2; }
bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ------------------------------------------------------------------------------------ measurement hooks
std::atomic<uint64_t> g_launches{0};
bool g_profile = false;
constexpr int kEventPool = 8192;
struct TimedLaunch {
    int kind;
    cudaEvent_t start, stop;
};
std::vector<TimedLaunch> g_timed;      // recorded launches since profiling was enabled
std::vector<cudaEvent_t> g_free_events;

cudaEvent_t take_event() {
    if (!g_free_events.empty()) {
        cudaEvent_t e = g_free_events.back();
        g_free_events.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

struct LaunchScope {
    cudaStream_t stream;
    bool timed = false;
    TimedLaunch rec{};
    LaunchScope(int kind, cudaStream_t s) : stream(s) {
        g_launches.fetch_add(1, std::memory_order_relaxed);
        if (g_profile && static_cast<int>(g_timed.size()) < kEventPool) {
            rec.kind = kind;
            rec.start = take_event();
            rec.stop = take_event();
            if (rec.start && rec.stop) {
                timed = true;
                cudaEventRecord(rec.start, stream);
            }
        }
    }
    ~LaunchScope() {
        if (timed) {
            cudaEventRecord(rec.stop, stream);
            g_timed.push_back(rec);
        }
    }
};

// ------------------------------------------------------------------------------------ planning
// How a streaming kernel covers `rows` rows of P positions: vector width, tiles per row, rows per block.
struct ColPlan {
    int V = 1;
    unsigned tiles = 0, TP = 0;
    int rows = 0, chunk = 0, nchunks = 0, max_slots = 0;
    unsigned grid() const { return tiles * static_cast<unsigned>(nchunks); }
    PartialLayout layout() const { return PartialLayout{nchunks, tiles, TP, max_slots}; }
    size_t partial_count() const { return static_cast<size_t>(nchunks) * tiles * max_slots; }
};

// Blocks per launch aimed at when splitting the rows; 0 = a multiple of the SM count (32 per SM for the
// streaming kernels, 8 per SM - one wave, all loads in flight - for the short statistics kernels).
int g_target_blocks = 0;
int g_min_chunk = 8;                      // ... but at least this many rows per block
int g_stat_target_blocks = 0;
int g_stat_min_chunk = 1;

int target_blocks_streaming() { return g_target_blocks > 0 ? g_target_blocks : sm_count() * 32; }
int target_blocks_statistics() { return g_stat_target_blocks > 0 ? g_stat_target_blocks : sm_count() * 8; }

// Full BN streams the whole tensor in three of its five kernels; on tensors of tens of MB it measured 5-8 %
// faster with blocks twice as long (fewer partials, fewer block prologues), the sampled rules did not.
int g_full_min_chunk = 16;
constexpr double kLongChunkBytes = 32.0 * 1048576.0;

ColPlan plan_col(unsigned P, int HW, int C, int rows, int ebytes, bool statistics = false, bool full_bn = false) {
    const int target_blocks = statistics ? target_blocks_statistics() : target_blocks_streaming();
    int min_chunk = statistics ? g_stat_min_chunk : g_min_chunk;
    if (full_bn && static_cast<double>(rows) * P * ebytes >= kLongChunkBytes) min_chunk = std::max(min_chunk, g_full_min_chunk);
    ColPlan pl;
    int V = 16 / ebytes;
    while (V > 1 && P % static_cast<unsigned>(V) != 0) V >>= 1;
    pl.V = V;
    pl.TP = static_cast<unsigned>(kThreads) * V;
    pl.tiles = (P + pl.TP - 1) / pl.TP;
    pl.rows = rows;
    // as many row chunks as keep the grid within the target (one wave of resident blocks)
    long want = target_blocks / static_cast<long>(pl.tiles);
    long nchunks = std::max(1L, std::min<long>(want, std::max(1, rows / min_chunk)));
    pl.chunk = static_cast<int>((rows + nchunks - 1) / nchunks);
    pl.nchunks = (rows + pl.chunk - 1) / pl.chunk;
    long slots = (static_cast<long>(pl.TP) + HW - 2) / HW + 1;
    pl.max_slots = static_cast<int>(std::min<long>(slots, C));
    return pl;
}

// Patch kernels: a sample row has C*ph*pw compact positions, 256 per block.
struct PatchPlan {
    unsigned tiles = 0;
    int chunk = 0, nchunks = 0, max_slots = 0;
    unsigned grid() const { return tiles * static_cast<unsigned>(nchunks); }
    PartialLayout layout() const { return PartialLayout{nchunks, tiles, static_cast<unsigned>(kThreads), max_slots}; }
    size_t partial_count() const { return static_cast<size_t>(nchunks) * tiles * max_slots; }
};

PatchPlan plan_patch(int N, int C, int ph, int pw) {
    PatchPlan pl;
    const long PP = static_cast<long>(ph) * pw;
    const long Pc = static_cast<long>(C) * PP;
    pl.tiles = static_cast<unsigned>((Pc + kThreads - 1) / kThreads);
    long want = target_blocks_statistics() / static_cast<long>(pl.tiles);
    long nchunks = std::max(1L, std::min<long>(want, std::max(1, N / 4)));
    pl.chunk = static_cast<int>((N + nchunks - 1) / nchunks);
    pl.nchunks = (N + pl.chunk - 1) / pl.chunk;
    pl.max_slots = static_cast<int>(std::min<long>((kThreads + PP - 2) / PP + 1, C));
    return pl;
}

// ------------------------------------------------------------------------------------ slab (on-chip) path
// A layer takes the one-launch path when the data of a channel group, split over the blocks of a
// cluster, fits their shared memory (see bns_slab_kernels.cuh).
struct SlabPlan {
    bool ok = false;
    SlabGeom geo{};
    unsigned grid = 0;
};

bool g_slab = true;            // use the one-launch path where it applies
int g_slab_cta_kb = 112;       // preferred shared memory per block: two blocks per SM stay resident
int g_slab_min_ctas = 0;       // grow the cluster while the launch has fewer blocks than this; 0 = 2 per SM
int g_slab_max_mb = 6;         // tensors larger than this many MiB keep the streaming path (measured: see bns.h)
int g_slab_cluster_max = 8;    // largest cluster (8 is the portable limit)
bool g_slab_small_sets = false;  // also for small sampled sets (whose streaming path is short already; measured slower)
constexpr size_t kSlabSmemLimit = 227 * 1024;  // most dynamic shared memory a block may ask for

size_t gcd_size(size_t a, size_t b) { return b ? gcd_size(b, a % b) : a; }

// Shared memory layout of one block for cluster size R; returns the total bytes.
size_t slab_layout(SlabGeom& g, int R, int tensors, int origin_stride) {
    auto up = [](size_t v, size_t a) { return (v + a - 1) / a * a; };
    g.R = R;
    g.rows_max = (g.N + R - 1) / R;
    const int K = 2;        // sums kept per position
    size_t off = 128;       // the copy barrier lives at offset 0
    g.off_x = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(g.rows_max) * g.row_bytes, 128);
    g.off_g = static_cast<unsigned>(off);
    if (tensors == 2) off = up(off + static_cast<size_t>(g.rows_max) * g.row_bytes, 128);
    g.off_fold = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(K) * g.RL * g.Wd * sizeof(float), 16);
    g.off_slices = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(std::max(g.G, kWarps)) * K * sizeof(float), 16);
    g.off_part = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(g.G) * 16, 16);
    g.off_all = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(R) * g.G * 16, 16);
    g.off_coef = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(g.G) * 16, 16);
    g.off_flag = static_cast<unsigned>(off);
    off = up(off + static_cast<size_t>(g.rows_max), 16);
    g.off_origin = static_cast<unsigned>(off);
    off = up(off + std::max<size_t>(16, static_cast<size_t>(g.rows_max) * origin_stride * sizeof(int2)), 16);
    g.total_bytes = static_cast<unsigned>(off);
    return off;
}

// Channel groups: the fewest channels whose row segment is a multiple of 16 bytes, doubled while the
// segment is shorter than 512 bytes.  False if the shape does not fit the scheme (a segment wider than
// kThreads vectors, or C not a multiple of the group).
bool group_geometry(int N, int C, int H, int W, int ebytes, SlabGeom& g) {
    const size_t HW = static_cast<size_t>(H) * W;
    if (H >= 32768 || W >= 65536) return false;
    const int V = 16 / ebytes;
    int G = static_cast<int>(16 / gcd_size(HW * ebytes, 16));
    if (C % G != 0) return false;
    while (static_cast<size_t>(G) * HW * ebytes < 512 && C % (2 * G) == 0 && 2 * G * HW / V <= static_cast<size_t>(kThreads) &&
           2 * G <= kSlabMaxChannels)
        G *= 2;
    if (G * HW / V > static_cast<size_t>(kThreads) || G > kSlabMaxChannels) return false;
    g = SlabGeom{};
    g.N = N;
    g.C = C;
    g.H = H;
    g.W = W;
    g.HW = static_cast<int>(HW);
    g.G = G;
    g.Wd = static_cast<int>(G * HW);
    g.NV = g.Wd / V;
    g.RL = kThreads / g.NV;
    g.P = static_cast<unsigned>(C * HW);
    g.row_bytes = static_cast<unsigned>(g.Wd * ebytes);
    return true;
}

// Sampled elements per channel up to which a sampled set counts as small: one block can read all of it.
int g_direct_max = 8192;

// origin_stride: 0 = no device-resident patch offsets, 1 = one pair per sample, 2 = one pair per map
SlabPlan plan_slab(int N, int C, int H, int W, int ebytes, bool backward, int offsets_kind) {
    SlabPlan sp;
    if (!g_slab) return sp;
    const size_t HW = static_cast<size_t>(H) * W;
    if (static_cast<double>(N) * C * HW * ebytes > static_cast<double>(g_slab_max_mb) * 1048576.0) return sp;
    if (!group_geometry(N, C, H, W, ebytes, sp.geo)) return sp;
    SlabGeom& g = sp.geo;
    const int G = g.G;
    const int tensors = backward ? 2 : 1;
    const int stride = offsets_kind == 2 ? G : offsets_kind == 1 ? 1 : 0;
    const int groups = C / G;
    const int r_max = std::min(g_slab_cluster_max, N);
    int R = 0;
    for (int limit_pass = 0; limit_pass < 2 && !R; ++limit_pass) {
        const size_t limit = limit_pass == 0 ? std::min(static_cast<size_t>(g_slab_cta_kb) * 1024, kSlabSmemLimit) : kSlabSmemLimit;
        for (int r = 1; r <= r_max; r *= 2)
            if (slab_layout(g, r, tensors, stride) <= limit) {
                R = r;
                break;
            }
    }
    if (!R) return sp;
    const int want = g_slab_min_ctas > 0 ? g_slab_min_ctas : 2 * sm_count();
    while (2 * R <= r_max && groups * R < want && N / (2 * R) >= 4) R *= 2;
    slab_layout(g, R, tensors, stride);
    sp.grid = static_cast<unsigned>(groups) * R;
    sp.ok = true;
    return sp;
}

struct Problem {
    int N, C, H, W, HW, dtype;
    unsigned P;
    size_t elems;
    int rule;
    // resolved sampling
    int count = 0;                 // BATCH: k; VIRTUAL: nv
    int begin = 0;                 // BATCH, contiguous ascending list: first index
    bool contiguous = true;        // BATCH: list is begin .. begin+k-1
    PatchRule patch{};
    double s = 0;                  // points per channel that enter the statistics
    // plans
    ColPlan main_plan;             // all N rows of x (normalise, backward pass 1, full statistics, full backward)
    ColPlan stat_plan;             // BATCH: the k sampled rows;  VIRTUAL: the nv rows of xv
    PatchPlan patch_plan;
    SlabPlan slab_fwd, slab_bwd;   // the one-launch on-chip path, when the layer qualifies
    // workspace layout
    size_t off_list, off_stats, off_bwd, off_bwd_v, total;
};

bns_status check_shape(const bns_shape* sh) {
    if (!sh) return BNS_ERR_NULL;
    if (sh->N <= 0 || sh->C <= 0 || sh->H <= 0 || sh->W <= 0) return BNS_ERR_SHAPE;
    if (sh->dtype != BNS_F32 && sh->dtype != BNS_BF16) return BNS_ERR_DTYPE;
    double P = static_cast<double>(sh->C) * sh->H * sh->W;
    if (P >= 2147483648.0) return BNS_ERR_SHAPE;              // positions of one sample are indexed with 32 bits
    if (static_cast<double>(sh->N) * sh->C >= 2147483648.0) return BNS_ERR_SHAPE;
    return BNS_OK;
}

// Validates everything that can be validated on the host and fills the plan.
bns_status make_problem(const bns_shape* sh, const bns_sampling* sp, Problem& pb) {
    bns_status st = check_shape(sh);
    if (st != BNS_OK) return st;
    if (!sp) return BNS_ERR_NULL;
    pb.N = sh->N;
    pb.C = sh->C;
    pb.H = sh->H;
    pb.W = sh->W;
    pb.HW = sh->H * sh->W;
    pb.dtype = sh->dtype;
    pb.P = static_cast<unsigned>(sh->C) * static_cast<unsigned>(pb.HW);
    pb.elems = static_cast<size_t>(pb.N) * pb.P;
    pb.rule = sp->rule;
    const int eb = elem_bytes(pb.dtype);
    pb.main_plan = plan_col(pb.P, pb.HW, pb.C, pb.N, eb, false, sp->rule == BNS_RULE_FULL);
    pb.stat_plan = pb.main_plan;
    switch (sp->rule) {
    case BNS_RULE_FULL:
        pb.s = static_cast<double>(pb.N) * pb.HW;
        break;
    case BNS_RULE_BATCH: {
        if (sp->k < 1 || sp->k > pb.N) return BNS_ERR_RULE;
        if (!sp->sample_idx) return BNS_ERR_NULL;
        std::vector<char> seen(pb.N, 0);
        pb.contiguous = true;
        for (int j = 0; j < sp->k; ++j) {
            int v = sp->sample_idx[j];
            if (v < 0 || v >= pb.N || seen[v]) return BNS_ERR_INDEX;
            seen[v] = 1;
            if (v != sp->sample_idx[0] + j) pb.contiguous = false;
        }
        pb.count = sp->k;
        pb.begin = sp->sample_idx[0];
        pb.s = static_cast<double>(sp->k) * pb.HW;
        pb.stat_plan = plan_col(pb.P, pb.HW, pb.C, sp->k, eb, true);
        break;
    }
    case BNS_RULE_FEATURE: {
        if (sp->ph < 1 || sp->ph > pb.H || sp->pw < 1 || sp->pw > pb.W) return BNS_ERR_RULE;
        if (sp->offset_mode < BNS_OFF_SHARED || sp->offset_mode > BNS_OFF_PER_MAP) return BNS_ERR_RULE;
        if (!sp->offsets) return BNS_ERR_NULL;
        pb.patch.ph = sp->ph;
        pb.patch.pw = sp->pw;
        if (sp->offset_mode == BNS_OFF_SHARED) {
            int oh = sp->offsets[0], ow = sp->offsets[1];
            if (oh < 0 || oh > pb.H - sp->ph || ow < 0 || ow > pb.W - sp->pw) return BNS_ERR_INDEX;
            pb.patch.oh = oh;
            pb.patch.ow = ow;
            pb.patch.offsets = nullptr;
        } else {
            if (reinterpret_cast<uintptr_t>(sp->offsets) & 7u) return BNS_ERR_ALIGN;
            pb.patch.offsets = sp->offsets;
            pb.patch.stride_n = sp->offset_mode == BNS_OFF_PER_SAMPLE ? 1 : pb.C;
            pb.patch.stride_c = sp->offset_mode == BNS_OFF_PER_SAMPLE ? 0 : 1;
        }
        pb.s = static_cast<double>(pb.N) * sp->ph * sp->pw;
        pb.patch_plan = plan_patch(pb.N, pb.C, sp->ph, sp->pw);
        break;
    }
    case BNS_RULE_VIRTUAL: {
        if (sp->nv < 1) return BNS_ERR_RULE;
        if (sp->xv_dtype != BNS_F32 && sp->xv_dtype != BNS_BF16) return BNS_ERR_DTYPE;
        if (!sp->xv) return BNS_ERR_NULL;
        if (!aligned16(sp->xv) || !aligned16(sp->yv) || !aligned16(sp->dyv) || !aligned16(sp->dxv)) return BNS_ERR_ALIGN;
        pb.count = sp->nv;
        pb.s = static_cast<double>(sp->nv) * pb.HW;
        pb.stat_plan = plan_col(pb.P, pb.HW, pb.C, sp->nv, elem_bytes(sp->xv_dtype), true);
        break;
    }
    default:
        return BNS_ERR_RULE;
    }
    // workspace: header | sample list | statistics partials | backward partials (real) | (virtual)
    size_t off = kHeaderBytes;
    pb.off_list = off;
    off += align_up(static_cast<size_t>(pb.N) * sizeof(int));
    pb.off_stats = off;
    size_t stat_partials = std::max(pb.main_plan.partial_count(), pb.stat_plan.partial_count());
    if (sp->rule == BNS_RULE_FEATURE)
        stat_partials = std::max(stat_partials, pb.patch_plan.partial_count());
    off += align_up(stat_partials * sizeof(float4));
    pb.off_bwd = off;
    off += align_up(pb.main_plan.partial_count() * sizeof(float2));
    pb.off_bwd_v = off;
    if (sp->rule == BNS_RULE_VIRTUAL) off += align_up(pb.stat_plan.partial_count() * sizeof(float2));
    pb.total = off;
    const int offsets_kind = (sp->rule == BNS_RULE_FEATURE && pb.patch.offsets) ? (pb.patch.stride_c ? 2 : 1) : 0;
    if (g_slab_small_sets || sp->rule == BNS_RULE_FULL || pb.s > static_cast<double>(g_direct_max)) {
        pb.slab_fwd = plan_slab(pb.N, pb.C, pb.H, pb.W, eb, false, offsets_kind);
        pb.slab_bwd = plan_slab(pb.N, pb.C, pb.H, pb.W, eb, true, offsets_kind);
    }
    return BNS_OK;
}

bns_status check_workspace(const Problem& pb, const void* ws, size_t bytes) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) || bytes < pb.total) return BNS_ERR_WORKSPACE;
    return BNS_OK;
}

template <typename T>
T* ws_at(void* ws, size_t off) {
    return reinterpret_cast<T*>(static_cast<char*>(ws) + off);
}

// Launch failures of the current call, on this host thread: every launch helper records the return code
// of its own cudaLaunchKernelEx, so an error that some other code left in the runtime is neither
// reported as ours nor cleared.
thread_local bool t_launch_failed = false;

void note_launch(cudaError_t err) {
    if (err != cudaSuccess) {
        t_launch_failed = true;
        cudaGetLastError();  // a failed launch leaves its error behind: take it back out
    }
}

bns_status last_error() {
    const bool failed = t_launch_failed;
    t_launch_failed = false;
    return failed ? BNS_ERR_CUDA : BNS_OK;
}

// Copies a non-contiguous sample list into the workspace; returns the device list or NULL.
bns_status stage_list(const Problem& pb, const bns_sampling* sp, void* ws, cudaStream_t stream, const int** list) {
    *list = nullptr;
    if (pb.rule != BNS_RULE_BATCH || pb.contiguous) return BNS_OK;
    int* dev = ws_at<int>(ws, pb.off_list);
    if (cudaMemcpyAsync(dev, sp->sample_idx, sizeof(int) * sp->k, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return BNS_ERR_CUDA;
    *list = dev;
    return BNS_OK;
}

bns_status clear_status(const Problem& pb, void* ws, cudaStream_t stream, unsigned** status) {
    *status = nullptr;
    if (pb.rule == BNS_RULE_FEATURE && pb.patch.offsets) {
        if (cudaMemsetAsync(ws, 0, sizeof(unsigned), stream) != cudaSuccess) return BNS_ERR_CUDA;
        *status = ws_at<unsigned>(ws, 0);
    }
    return BNS_OK;
}

// ------------------------------------------------------------------------------------ launches
bool g_pdl = true;    // ask for programmatic dependent launch (blocks may be scheduled while the previous kernel drains)
bool g_fold_finalize = true;  // let the second backward pass finish the sums of Eq. 5 itself where it can
bool g_l2_order = true;  // order rows so that a kernel re-reads what the previous one left in L2

template <typename... KArgs, typename... Args>
void launch_with(bool early_scheduling, int kind, void (*kernel)(KArgs...), unsigned grid, cudaStream_t s,
                 Args&&... args) {
    LaunchScope scope(kind, s);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (g_pdl && early_scheduling) ? 1 : 0;
    note_launch(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

// Normal launch of this library: the kernel may be scheduled while its predecessor drains.
template <typename... KArgs, typename... Args>
void launch(int kind, void (*kernel)(KArgs...), unsigned grid, cudaStream_t s, Args&&... args) {
    launch_with(true, kind, kernel, grid, s, static_cast<Args&&>(args)...);
}

// For a kernel that touches its inputs before its dependency wait and is the first kernel of a call:
// whatever precedes it in the stream may have produced those inputs, so it must not start early.
template <typename... KArgs, typename... Args>
void launch_after_predecessor(int kind, void (*kernel)(KArgs...), unsigned grid, cudaStream_t s, Args&&... args) {
    launch_with(false, kind, kernel, grid, s, static_cast<Args&&>(args)...);
}

#define BNS_BY_TYPE_V(dtype, V_, CALL)                   \
    do {                                                 \
        if ((dtype) == BNS_F32) {                        \
            using T = F32;                               \
            switch (V_) {                                \
            case 4: { constexpr int V = 4; CALL; } break; \
            case 2: { constexpr int V = 2; CALL; } break; \
            default: { constexpr int V = 1; CALL; } break; \
            }                                            \
        } else {                                         \
            using T = BF16;                              \
            switch (V_) {                                \
            case 8: { constexpr int V = 8; CALL; } break; \
            case 4: { constexpr int V = 4; CALL; } break; \
            case 2: { constexpr int V = 2; CALL; } break; \
            default: { constexpr int V = 1; CALL; } break; \
            }                                            \
        }                                                \
    } while (0)

#define BNS_BY_TYPE(dtype, CALL)   \
    do {                           \
        if ((dtype) == BNS_F32) {  \
            using T = F32;         \
            CALL;                  \
        } else {                   \
            using T = BF16;        \
            CALL;                  \
        }                          \
    } while (0)

template <typename T>
const typename T::storage* in(const void* p) {
    return static_cast<const typename T::storage*>(p);
}
template <typename T>
typename T::storage* out(void* p) {
    return static_cast<typename T::storage*>(p);
}

// Backward pass 1 keeps its sums per channel where the maps are large and per position where they are
// small (see col_bwd_reduce_kernel); one element per thread always takes the per-position form.
int g_per_channel_min_hw = 512;

template <typename T, int V, bool WRITE_DX>
auto bwd_reduce_variant(int HW) -> decltype(&col_bwd_reduce_kernel<T, V, WRITE_DX, false>) {
    if constexpr (V >= 2) {
        if (HW >= V && HW >= g_per_channel_min_hw) return col_bwd_reduce_kernel<T, V, WRITE_DX, true>;
    }
    return col_bwd_reduce_kernel<T, V, WRITE_DX, false>;
}

unsigned warp_per_channel_grid(int C) { return static_cast<unsigned>((C + kThreads / 32 - 1) / (kThreads / 32)); }

// Small sampled sets are handled by one block per channel (no partials, no finalize launch).
bool small_sampled_set(const Problem& pb) { return pb.rule != BNS_RULE_FULL && pb.s <= static_cast<double>(g_direct_max); }

// The one-block-per-channel kernels come in two depths.  With more than kUnroll elements per thread and few
// enough channels for all blocks to be resident at the larger register count, a thread keeps kDirectUnroll
// loads in flight: fewer dependent trips to memory (CIFAR sweep 53 -> 48 us per step).  With more channels the
// lost occupancy costs more than that (256x512x28x28, 3x3 patches: second pass 28.6 -> 34.7 us).
bool deep_direct(const Problem& pb, const SampleSet& set) {
    return set.s > kUnroll * kThreads && pb.C <= 2 * sm_count();
}

SampleSet sample_set(const Problem& pb, const int* list) {
    SampleSet set{};
    set.patches = pb.rule == BNS_RULE_FEATURE;
    set.list = list;
    set.begin = pb.rule == BNS_RULE_BATCH ? pb.begin : 0;
    set.rows = pb.count;
    set.patch = pb.patch;
    set.N = pb.N;
    set.C = pb.C;
    set.H = pb.H;
    set.W = pb.W;
    set.s = static_cast<int>(pb.s);
    return set;
}

// Launch of a slab kernel: a cluster of `cluster` blocks per channel group and `smem` bytes of dynamic
// shared memory per block.  The first launch of each kernel on a device raises its shared-memory limit.
std::mutex g_slab_attr_mutex;

template <typename... KArgs, typename... Args>
void launch_cluster(int kind, void (*kernel)(KArgs...), unsigned grid, unsigned cluster, size_t smem, cudaStream_t s,
                    Args&&... args) {
    if (smem > 48 * 1024) {
        static bool raised[kMaxDevices] = {};  // one array per kernel instantiation
        int device = -1;
        if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= kMaxDevices) {
            note_launch(cudaErrorInvalidDevice);
            return;
        }
        std::lock_guard<std::mutex> guard(g_slab_attr_mutex);
        if (!raised[device]) {
            if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSlabSmemLimit)) !=
                cudaSuccess) {
                note_launch(cudaErrorInvalidValue);
                return;
            }
            raised[device] = true;
        }
    }
    LaunchScope scope(kind, s);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = cluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_pdl ? 2 : 1;
    note_launch(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

SlabSel slab_selection(const Problem& pb, const bns_sampling* sp, const int* list) {
    SlabSel sel{};
    sel.rule = pb.rule;
    sel.list = list;
    sel.begin = pb.rule == BNS_RULE_BATCH ? pb.begin : 0;
    sel.count = pb.count;
    sel.patch = pb.patch;
    sel.inv_s = static_cast<float>(1.0 / pb.s);
    if (pb.rule == BNS_RULE_VIRTUAL) {
        sel.nv = sp->nv;
        sel.xv_is_bf16 = sp->xv_dtype == BNS_BF16;
        sel.xv = sp->xv;
        sel.yv = sp->yv;
        sel.dyv = sp->dyv;
        sel.dxv = sp->dxv;
    }
    return sel;
}

bns_status slab_forward(const Problem& pb, const bns_sampling* sp, const void* x, const float* gamma, const float* beta,
                        float eps, void* y, float* mean, float* invstd, void* ws, cudaStream_t stream,
                        const MovingAverage& ma) {
    unsigned* status;
    bns_status st = clear_status(pb, ws, stream, &status);
    if (st != BNS_OK) return st;
    const int* list = nullptr;
    st = stage_list(pb, sp, ws, stream, &list);
    if (st != BNS_OK) return st;
    const SlabPlan& pl = pb.slab_fwd;
    const SlabSel sel = slab_selection(pb, sp, list);
    BNS_BY_TYPE(pb.dtype, (launch_cluster(BNS_KERNEL_SLAB_FORWARD, slab_forward_kernel<T>, pl.grid, pl.geo.R,
                                          pl.geo.total_bytes, stream, in<T>(x), out<T>(y), gamma, beta, eps, pl.geo, sel, mean,
                                          invstd, status, ma)));
    return last_error();
}

bns_status slab_backward(const Problem& pb, const bns_sampling* sp, const void* x, const void* dy, const float* gamma,
                         const float* mean, const float* invstd, void* dx, float* dgamma, float* dbeta, void* ws,
                         cudaStream_t stream) {
    unsigned* status;
    bns_status st = clear_status(pb, ws, stream, &status);
    if (st != BNS_OK) return st;
    const int* list = nullptr;
    st = stage_list(pb, sp, ws, stream, &list);
    if (st != BNS_OK) return st;
    const SlabPlan& pl = pb.slab_bwd;
    const SlabSel sel = slab_selection(pb, sp, list);
    BNS_BY_TYPE(pb.dtype, (launch_cluster(BNS_KERNEL_SLAB_BACKWARD, slab_backward_kernel<T>, pl.grid, pl.geo.R,
                                          pl.geo.total_bytes, stream, in<T>(x), in<T>(dy), out<T>(dx), gamma, mean, invstd,
                                          pl.geo, sel, dgamma, dbeta, status)));
    return last_error();
}

// Statistics of the rule's sampled set into mean / invstd: partial moments, then one warp per channel.
// `virtual_out` (with gamma, beta): under the VIRTUAL rule with a small set, the kernel that takes the
// statistics also writes the normalised virtual samples there and *virtual_done is set.
bns_status run_statistics(const Problem& pb, const bns_sampling* sp, const void* x, float eps, float* mean,
                          float* invstd, void* ws, cudaStream_t stream, const MovingAverage& ma = MovingAverage{},
                          void* virtual_out = nullptr, const float* gamma = nullptr, const float* beta = nullptr,
                          bool* virtual_done = nullptr) {
    if (small_sampled_set(pb)) {
        unsigned* status;
        bns_status st = clear_status(pb, ws, stream, &status);
        if (st != BNS_OK) return st;
        const int* list = nullptr;
        st = stage_list(pb, sp, ws, stream, &list);
        if (st != BNS_OK) return st;
        const SampleSet set = sample_set(pb, list);
        const void* data = pb.rule == BNS_RULE_VIRTUAL ? sp->xv : x;
        const int dt = pb.rule == BNS_RULE_VIRTUAL ? sp->xv_dtype : pb.dtype;
        if (deep_direct(pb, set))
            BNS_BY_TYPE(dt, (launch(BNS_KERNEL_DIRECT_MOMENTS, direct_moments_kernel<T, kDirectUnroll>,
                                    static_cast<unsigned>(pb.C), stream, in<T>(data), set, eps, mean, invstd, status, ma,
                                    out<T>(pb.rule == BNS_RULE_VIRTUAL ? virtual_out : nullptr), gamma, beta)));
        else
            BNS_BY_TYPE(dt, (launch(BNS_KERNEL_DIRECT_MOMENTS, direct_moments_kernel<T>, static_cast<unsigned>(pb.C), stream,
                                    in<T>(data), set, eps, mean, invstd, status, ma,
                                    out<T>(pb.rule == BNS_RULE_VIRTUAL ? virtual_out : nullptr), gamma, beta)));
        if (virtual_done && pb.rule == BNS_RULE_VIRTUAL && virtual_out) *virtual_done = true;
        return last_error();
    }
    StatsSink sink{ws_at<float4>(ws, pb.off_stats), PartialLayout{}, static_cast<float>(1.0 / pb.s), eps, mean, invstd, ma};
    int span = pb.HW;  // positions per channel in the producer's position space
    if (pb.rule == BNS_RULE_FEATURE) {
        unsigned* status;
        bns_status st = clear_status(pb, ws, stream, &status);
        if (st != BNS_OK) return st;
        const PatchPlan& pp = pb.patch_plan;
        sink.L = pp.layout();
        span = pb.patch.ph * pb.patch.pw;
        BNS_BY_TYPE(pb.dtype, (launch(BNS_KERNEL_PATCH_MOMENTS, patch_moments_kernel<T>, pp.grid(), stream, in<T>(x),
                                      pb.patch, pb.N, pb.C, pb.H, pb.W, pp.nchunks, pp.tiles, sink, status)));
    } else {
        const int* list = nullptr;
        bns_status st = stage_list(pb, sp, ws, stream, &list);
        if (st != BNS_OK) return st;
        const ColPlan& pl = pb.rule == BNS_RULE_FULL ? pb.main_plan : pb.stat_plan;
        const void* data = pb.rule == BNS_RULE_VIRTUAL ? sp->xv : x;
        const int dt = pb.rule == BNS_RULE_VIRTUAL ? sp->xv_dtype : pb.dtype;
        const int begin = pb.rule == BNS_RULE_BATCH ? pb.begin : 0;
        sink.L = pl.layout();
        BNS_BY_TYPE_V(dt, pl.V,
                      (launch(BNS_KERNEL_COL_MOMENTS, col_moments_kernel<T, V>, pl.grid(), stream, in<T>(data), list, begin,
                              pl.rows, pl.nchunks, pl.tiles, pb.HW, pb.P, sink)));
    }
    launch(BNS_KERNEL_FINALIZE_STATS, finalize_stats_kernel, warp_per_channel_grid(pb.C), stream, sink, pb.C, span);
    return last_error();
}

bns_status forward_impl(const Problem& pb, const bns_sampling* sp, const void* x, const float* gamma, const float* beta,
                        float eps, void* y, float* mean, float* invstd, void* ws, cudaStream_t stream,
                        const MovingAverage& ma = MovingAverage{}) {
    if (pb.slab_fwd.ok) return slab_forward(pb, sp, x, gamma, beta, eps, y, mean, invstd, ws, stream, ma);
    bool virtual_done = false;
    bns_status st = run_statistics(pb, sp, x, eps, mean, invstd, ws, stream, ma,
                                   pb.rule == BNS_RULE_VIRTUAL ? sp->yv : nullptr, gamma, beta, &virtual_done);
    if (st != BNS_OK) return st;
    const ColPlan& pl = pb.main_plan;
    // The few virtual samples go first (unless the statistics kernel has normalised them already): that short
    // kernel then runs while the blocks of the large one that follows are being scheduled and requesting
    // their first rows.
    if (pb.rule == BNS_RULE_VIRTUAL && sp->yv && !virtual_done) {
        const ColPlan& pv = pb.stat_plan;
        BNS_BY_TYPE_V(sp->xv_dtype, pv.V,
                      (launch(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pv.grid(), stream, in<T>(sp->xv),
                              out<T>(sp->yv), gamma, beta, mean, invstd, RowOrder{RowOrder::kIdentity, pv.rows, 0, 0},
                              pv.nchunks, pv.tiles, pb.HW, pb.P)));
    }
    // visit first the rows that the statistics kernel has just read: they are still in L2
    RowOrder order{RowOrder::kIdentity, pb.N, 0, 0};
    if (g_l2_order && pb.rule == BNS_RULE_FULL) order.mode = RowOrder::kReversed;
    if (g_l2_order && pb.rule == BNS_RULE_BATCH && pb.contiguous)
        order = RowOrder{RowOrder::kRangeFirst, pb.N, pb.begin, pb.count};
    BNS_BY_TYPE_V(pb.dtype, pl.V,
                  (launch(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pl.grid(), stream, in<T>(x), out<T>(y), gamma,
                          beta, mean, invstd, order, pl.nchunks, pl.tiles, pb.HW, pb.P)));
    return last_error();
}

bns_status backward_impl(const Problem& pb, const bns_sampling* sp, const void* x, const void* dy, const float* gamma,
                         const float* mean, const float* invstd, void* dx, float* dgamma, float* dbeta, void* ws,
                         cudaStream_t stream) {
    if (pb.slab_bwd.ok) return slab_backward(pb, sp, x, dy, gamma, mean, invstd, dx, dgamma, dbeta, ws, stream);
    const ColPlan& pl = pb.main_plan;
    const ColPlan& pv = pb.stat_plan;
    const bool full = pb.rule == BNS_RULE_FULL;
    const bool virtual_grads = pb.rule == BNS_RULE_VIRTUAL && sp->dyv;
    GradSink sink{ws_at<float2>(ws, pb.off_bwd), pl.layout(), virtual_grads ? ws_at<float2>(ws, pb.off_bwd_v) : nullptr,
                  pv.layout(), invstd, dgamma, dbeta};
    // pass 1: the sums of Eq. 5 over every real element; dx = gamma invstd dy everywhere unless every
    // element is sampled (FULL), where the second pass writes dx anyway.  The rows that the second pass
    // reads again are visited last, so that it finds them in L2.
    RowOrder order{RowOrder::kIdentity, pb.N, 0, 0};
    if (g_l2_order && pb.rule == BNS_RULE_BATCH && pb.contiguous)
        order = RowOrder{RowOrder::kRangeLast, pb.N, pb.begin, pb.count};
    if (full)
        BNS_BY_TYPE_V(pb.dtype, pl.V,
                      (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, false>(pb.HW), pl.grid(), stream, in<T>(x),
                              in<T>(dy), out<T>(nullptr), gamma, mean, invstd, order, pl.nchunks, pl.tiles, pb.HW, pb.P,
                              false, sink)));
    else
        BNS_BY_TYPE_V(pb.dtype, pl.V,
                      (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, true>(pb.HW), pl.grid(), stream, in<T>(x),
                              in<T>(dy), out<T>(dx), gamma, mean, invstd, order, pl.nchunks, pl.tiles, pb.HW, pb.P, false,
                              sink)));
    if (virtual_grads)
        BNS_BY_TYPE_V(sp->xv_dtype, pv.V,
                      (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, false>(pb.HW), pv.grid(), stream, in<T>(sp->xv),
                              in<T>(sp->dyv), out<T>(nullptr), gamma, mean, invstd,
                              RowOrder{RowOrder::kIdentity, pv.rows, 0, 0}, pv.nchunks, pv.tiles, pb.HW, pb.P, true,
                              sink)));
    if (small_sampled_set(pb)) {
        // one block per channel combines the channel's sums and applies the statistics terms to its sampled set
        unsigned* status;
        bns_status st = clear_status(pb, ws, stream, &status);
        if (st != BNS_OK) return st;
        const int* list = nullptr;
        st = stage_list(pb, sp, ws, stream, &list);
        if (st != BNS_OK) return st;
        const SampleSet set = sample_set(pb, list);
        const bool deep = deep_direct(pb, set);
        if (pb.rule == BNS_RULE_VIRTUAL && deep)
            BNS_BY_TYPE(sp->xv_dtype,
                        (launch(BNS_KERNEL_DIRECT_FIXUP, direct_finalize_fixup_kernel<T, kDirectUnroll>,
                                static_cast<unsigned>(pb.C), stream, in<T>(sp->xv), in<T>(sp->dyv), out<T>(sp->dxv), gamma,
                                mean, sink, pb.HW, set, status)));
        else if (pb.rule == BNS_RULE_VIRTUAL)
            BNS_BY_TYPE(sp->xv_dtype,
                        (launch(BNS_KERNEL_DIRECT_FIXUP, direct_finalize_fixup_kernel<T>, static_cast<unsigned>(pb.C),
                                stream, in<T>(sp->xv), in<T>(sp->dyv), out<T>(sp->dxv), gamma, mean, sink, pb.HW, set,
                                status)));
        else if (deep)
            BNS_BY_TYPE(pb.dtype,
                        (launch(BNS_KERNEL_DIRECT_FIXUP, direct_finalize_fixup_kernel<T, kDirectUnroll>,
                                static_cast<unsigned>(pb.C), stream, in<T>(x), in<T>(dy), out<T>(dx), gamma, mean, sink,
                                pb.HW, set, status)));
        else
            BNS_BY_TYPE(pb.dtype,
                        (launch(BNS_KERNEL_DIRECT_FIXUP, direct_finalize_fixup_kernel<T>, static_cast<unsigned>(pb.C),
                                stream, in<T>(x), in<T>(dy), out<T>(dx), gamma, mean, sink, pb.HW, set, status)));
        return last_error();
    }
    // pass 2: the statistics terms, on S only.  Where a tile of the second pass meets few channels, its kernel
    // finishes the sums of Eq. 5 itself (every block re-adds the partials of its channels in the same fixed
    // order, one block per channel publishes dgamma / dbeta); otherwise a finalize launch comes first.
    const bool has_second_pass = pb.rule != BNS_RULE_VIRTUAL || sp->dxv;
    const int second_pass_slots = pb.rule == BNS_RULE_FEATURE ? pb.patch_plan.max_slots
                                  : pb.rule == BNS_RULE_FULL  ? pl.max_slots
                                                              : pv.max_slots;
    // (not for full BN: its second pass is a stream over the whole tensor, whose many short-lived blocks would each
    // pay the latency of re-adding the partials before their first load - measured 3 % slower)
    const int fold = g_fold_finalize && !full && has_second_pass && second_pass_slots <= kFoldSlots ? 1 : 0;
    if (!fold) launch(BNS_KERNEL_FINALIZE_BWD, finalize_bwd_kernel, warp_per_channel_grid(pb.C), stream, sink, pb.C, pb.HW);
    const float inv_s = static_cast<float>(1.0 / pb.s);
    switch (pb.rule) {
    case BNS_RULE_FULL:
        BNS_BY_TYPE_V(pb.dtype, pl.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pl.grid(), stream, in<T>(x), in<T>(dy),
                              out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, static_cast<const int*>(nullptr), 0,
                              RowOrder{g_l2_order ? RowOrder::kReversed : RowOrder::kIdentity, pl.rows, 0, 0}, pl.nchunks,
                              pl.tiles, pb.HW, pb.P, sink, fold)));
        break;
    case BNS_RULE_BATCH: {
        const int* list = nullptr;
        bns_status st = stage_list(pb, sp, ws, stream, &list);
        if (st != BNS_OK) return st;
        BNS_BY_TYPE_V(pb.dtype, pv.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pv.grid(), stream, in<T>(x), in<T>(dy),
                              out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, list, pb.begin,
                              RowOrder{RowOrder::kIdentity, pv.rows, 0, 0}, pv.nchunks, pv.tiles, pb.HW, pb.P, sink, fold)));
        break;
    }
    case BNS_RULE_FEATURE: {
        unsigned* status;
        bns_status st = clear_status(pb, ws, stream, &status);
        if (st != BNS_OK) return st;
        const PatchPlan& pp = pb.patch_plan;
        BNS_BY_TYPE(pb.dtype, (launch(BNS_KERNEL_PATCH_FIXUP, patch_fixup_kernel<T>, pp.grid(), stream, in<T>(x), in<T>(dy),
                                      out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, pb.patch, pb.N, pb.C, pb.H,
                                      pb.W, pp.nchunks, pp.tiles, status, sink, fold)));
        break;
    }
    case BNS_RULE_VIRTUAL:
        if (sp->dxv)
            BNS_BY_TYPE_V(sp->xv_dtype, pv.V,
                          (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pv.grid(), stream, in<T>(sp->xv),
                                  in<T>(sp->dyv), out<T>(sp->dxv), gamma, mean, invstd, dgamma, dbeta, inv_s,
                                  static_cast<const int*>(nullptr), 0, RowOrder{RowOrder::kIdentity, pv.rows, 0, 0},
                                  pv.nchunks, pv.tiles, pb.HW, pb.P, sink, fold)));
        break;
    }
    return last_error();
}

// ------------------------------------------------------------------------------------ Eq. 4: VDN combined with a sampling rule
// Two problems over the same shape: the sampling rule of the real batch (BATCH or FEATURE) and the
// virtual samples.  Workspace: [rule's workspace | virtual workspace | 2 C floats].
struct MixedProblem {
    Problem real, virt;
    bns_sampling virt_rule;
    size_t off_virt, off_vec, total;
};

bns_status make_mixed(const bns_shape* sh, const bns_sampling* sp, float mix, MixedProblem& mp) {
    if (!sp) return BNS_ERR_NULL;
    if (sp->rule != BNS_RULE_BATCH && sp->rule != BNS_RULE_FEATURE) return BNS_ERR_RULE;
    if (!(mix >= 0.f && mix <= 1.f)) return BNS_ERR_RULE;
    bns_status st = make_problem(sh, sp, mp.real);
    if (st != BNS_OK) return st;
    mp.virt_rule = *sp;
    mp.virt_rule.rule = BNS_RULE_VIRTUAL;
    st = make_problem(sh, &mp.virt_rule, mp.virt);
    if (st != BNS_OK) return st;
    mp.off_virt = align_up(mp.real.total);
    mp.off_vec = mp.off_virt + align_up(mp.virt.total);
    mp.total = mp.off_vec + align_up(2 * static_cast<size_t>(mp.real.C) * sizeof(float));
    return BNS_OK;
}

unsigned per_channel_grid(int C) { return static_cast<unsigned>((C + kThreads - 1) / kThreads); }

bns_status forward_mixed_impl(const MixedProblem& mp, const bns_sampling* sp, const void* x, const float* gamma,
                              const float* beta, float eps, float mix, void* y, float* mean, float* invstd,
                              float* mean_s, float* mean_v, void* ws, cudaStream_t stream) {
    const Problem& pr = mp.real;
    const Problem& pv = mp.virt;
    void* ws_v = static_cast<char*>(ws) + mp.off_virt;
    float* invstd_s = ws_at<float>(ws, mp.off_vec);
    float* invstd_v = invstd_s + pr.C;
    bns_status st = run_statistics(pr, sp, x, eps, mean_s, invstd_s, ws, stream);        // Eq. 3 on the sampled real set
    if (st != BNS_OK) return st;
    st = run_statistics(pv, &mp.virt_rule, x, eps, mean_v, invstd_v, ws_v, stream);      // Eq. 3 on the virtual set
    if (st != BNS_OK) return st;
    launch(BNS_KERNEL_VECTOR, mix_stats_kernel, per_channel_grid(pr.C), stream, mean_s, invstd_s, mean_v, invstd_v, mix,
           pr.C, mean, invstd);                                                           // Eq. 4
    const ColPlan& pl = pr.main_plan;
    BNS_BY_TYPE_V(pr.dtype, pl.V,
                  (launch(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pl.grid(), stream, in<T>(x), out<T>(y), gamma,
                          beta, mean, invstd, RowOrder{RowOrder::kIdentity, pr.N, 0, 0}, pl.nchunks, pl.tiles, pr.HW,
                          pr.P)));
    if (sp->yv) {
        const ColPlan& pq = pv.stat_plan;
        BNS_BY_TYPE_V(sp->xv_dtype, pq.V,
                      (launch(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pq.grid(), stream, in<T>(sp->xv),
                              out<T>(sp->yv), gamma, beta, mean, invstd, RowOrder{RowOrder::kIdentity, pq.rows, 0, 0},
                              pq.nchunks, pq.tiles, pr.HW, pr.P)));
    }
    return last_error();
}

bns_status backward_mixed_impl(const MixedProblem& mp, const bns_sampling* sp, const void* x, const void* dy,
                               const float* gamma, const float* mean, const float* invstd, const float* mean_s,
                               const float* mean_v, float mix, void* dx, float* dgamma, float* dbeta, void* ws,
                               cudaStream_t stream) {
    const Problem& pr = mp.real;
    const Problem& pv = mp.virt;
    void* ws_v = static_cast<char*>(ws) + mp.off_virt;
    const ColPlan& pl = pr.main_plan;
    const ColPlan& pq = pv.stat_plan;
    GradSink sink{ws_at<float2>(ws, pr.off_bwd), pl.layout(), sp->dyv ? ws_at<float2>(ws_v, pv.off_bwd_v) : nullptr,
                  pq.layout(), invstd, dgamma, dbeta};
    // the sums of Eq. 5 over the real batch (and dx without the statistics terms), then over the virtual rows
    BNS_BY_TYPE_V(pr.dtype, pl.V,
                  (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, true>(pr.HW), pl.grid(), stream, in<T>(x), in<T>(dy),
                          out<T>(dx), gamma, mean, invstd, RowOrder{RowOrder::kIdentity, pr.N, 0, 0}, pl.nchunks, pl.tiles,
                          pr.HW, pr.P, false, sink)));
    if (sp->dyv)
        BNS_BY_TYPE_V(sp->xv_dtype, pq.V,
                      (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, false>(pr.HW), pq.grid(), stream, in<T>(sp->xv),
                              in<T>(sp->dyv), out<T>(nullptr), gamma, mean, invstd,
                              RowOrder{RowOrder::kIdentity, pq.rows, 0, 0}, pq.nchunks, pq.tiles, pr.HW, pr.P, true,
                              sink)));
    launch(BNS_KERNEL_FINALIZE_BWD, finalize_bwd_kernel, warp_per_channel_grid(pr.C), stream, sink, pr.C, pr.HW);
    // statistics terms on the sampled real set: share (1-mix) of dl/dE and dl/dVar, spread over s_s
    // elements, deviations taken about that set's own mean
    const float w_s = static_cast<float>((1.0 - static_cast<double>(mix)) / pr.s);
    if (pr.rule == BNS_RULE_BATCH) {
        const int* list = nullptr;
        bns_status st = stage_list(pr, sp, ws, stream, &list);
        if (st != BNS_OK) return st;
        const ColPlan& ps = pr.stat_plan;
        BNS_BY_TYPE_V(pr.dtype, ps.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, ps.grid(), stream, in<T>(x), in<T>(dy),
                              out<T>(dx), gamma, mean_s, invstd, dgamma, dbeta, w_s, list, pr.begin,
                              RowOrder{RowOrder::kIdentity, ps.rows, 0, 0}, ps.nchunks, ps.tiles, pr.HW, pr.P, GradSink{}, 0)));
    } else {
        unsigned* status;
        bns_status st = clear_status(pr, ws, stream, &status);
        if (st != BNS_OK) return st;
        const PatchPlan& pp = pr.patch_plan;
        BNS_BY_TYPE(pr.dtype, (launch(BNS_KERNEL_PATCH_FIXUP, patch_fixup_kernel<T>, pp.grid(), stream, in<T>(x), in<T>(dy),
                                      out<T>(dx), gamma, mean_s, invstd, dgamma, dbeta, w_s, pr.patch, pr.N, pr.C, pr.H,
                                      pr.W, pp.nchunks, pp.tiles, status, GradSink{}, 0)));
    }
    // and on the virtual samples: share mix, spread over s_v elements, about the virtual mean
    if (sp->dxv) {
        const float w_v = static_cast<float>(static_cast<double>(mix) / pv.s);
        BNS_BY_TYPE_V(sp->xv_dtype, pq.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pq.grid(), stream, in<T>(sp->xv),
                              in<T>(sp->dyv), out<T>(sp->dxv), gamma, mean_v, invstd, dgamma, dbeta, w_v,
                              static_cast<const int*>(nullptr), 0, RowOrder{RowOrder::kIdentity, pq.rows, 0, 0},
                              pq.nchunks, pq.tiles, pr.HW, pr.P, GradSink{}, 0)));
    }
    return last_error();
}

// ------------------------------------------------------------------------------------ channels-last (NHWC)
int g_nhwc_blocks = 0;  // blocks per channels-last launch; 0 = 8 per SM

struct NhwcLaunch {
    NhwcShape shape;
    dim3 grid;
    size_t partial_count() const { return static_cast<size_t>(grid.x) * shape.C; }
};

// Block shape and grid for visiting `total` rows of C channels.
NhwcLaunch plan_nhwc(int C, int ebytes, long total, bool statistics, bool no_partials = false) {
    NhwcLaunch l{};
    int V = 16 / ebytes;
    while (V > 1 && C % V != 0) V >>= 1;
    NhwcShape& s = l.shape;
    s.C = C;
    s.V_unused = V;
    s.CV = C / V;
    s.CW = std::min(s.CV, kThreads);
    s.RL = kThreads / s.CW;
    const int gy = (s.CV + s.CW - 1) / s.CW;
    // few, long-lived blocks: every block leaves one partial per channel, so the block count is also the
    // number of partials the finalize kernels have to read per channel
    (void)statistics;
    // (a pass that leaves no partials - normalise - takes four times as many, shorter-lived blocks: measured 70 -> 64 us
    // on 256x56x56x64 fp32.  Fewer blocks for the passes that do leave partials - four per SM - ran the ResNet-50 shapes
    // 5 % faster, but then a thread adds up so many rows that the fp32 sums of the backward left the absolute
    // tolerance on channels with a gradient near zero; compensated sums in double precision cost what was gained.)
    const long blocks = static_cast<long>(g_nhwc_blocks > 0 ? g_nhwc_blocks : sm_count() * 8) * (no_partials ? 4 : 1);
    const long target = std::max(1L, blocks / gy);
    long rpb = std::max<long>(static_cast<long>(s.RL) * kUnroll * 2, (total + target - 1) / target);
    rpb = (rpb + s.RL - 1) / s.RL * s.RL;
    s.rows_per_block = static_cast<int>(rpb);
    l.grid = dim3(static_cast<unsigned>(std::max(1L, (total + rpb - 1) / rpb)), static_cast<unsigned>(gy), 1);
    return l;
}

int nhwc_vector(int C, int ebytes) {
    int V = 16 / ebytes;
    while (V > 1 && C % V != 0) V >>= 1;
    return V;
}

// Small sampled sets: one block per strip of one or two channel-vectors visits every sampled row.
NhwcLaunch plan_nhwc_direct(int C, int ebytes, long total) {
    NhwcLaunch l{};
    int V = 16 / ebytes;
    while (V > 1 && C % V != 0) V >>= 1;
    NhwcShape& s = l.shape;
    s.C = C;
    s.V_unused = V;
    s.CV = C / V;
    s.CW = std::min(s.CV, 2);
    s.RL = kThreads / s.CW;
    s.rows_per_block = static_cast<int>((total + s.RL - 1) / s.RL * s.RL);
    l.grid = dim3(1, static_cast<unsigned>((s.CV + s.CW - 1) / s.CW), 1);
    return l;
}

struct NhwcProblem {
    Problem pb;                  // shape and rule, validated as for NCHW
    long rows;                   // N*H*W
    long sampled_rows;           // rows in the sampled set (of x, or of xv for VIRTUAL)
    NhwcLaunch main, stat, virt; // all rows of x; the sampled rows; all rows of xv
    NhwcLaunch norm, norm_virt;  // the same rows as main / virt for the normalise pass, which leaves no partials
    NhwcLaunch direct;           // the sampled rows, one block per strip of channels (small sets)
    bool small_set = false;      // few enough sampled rows for `direct`
    size_t off_list, off_stats, off_bwd, off_bwd_v, total;
};

bns_status make_nhwc(const bns_shape* sh, const bns_sampling* sp, NhwcProblem& np) {
    bns_status st = make_problem(sh, sp, np.pb);
    if (st != BNS_OK) return st;
    const Problem& pb = np.pb;
    if (pb.rule == BNS_RULE_FEATURE && sp->offset_mode == BNS_OFF_PER_MAP) return BNS_ERR_RULE;  // a row spans all channels
    np.rows = static_cast<long>(pb.N) * pb.HW;
    if (np.rows >= 2147483647L) return BNS_ERR_SHAPE;
    const int eb = elem_bytes(pb.dtype);
    np.main = plan_nhwc(pb.C, eb, np.rows, false);
    np.norm = plan_nhwc(pb.C, eb, np.rows, false, true);
    np.virt = np.main;
    np.norm_virt = np.norm;
    switch (pb.rule) {
    case BNS_RULE_FULL: np.sampled_rows = np.rows; break;
    case BNS_RULE_BATCH: np.sampled_rows = static_cast<long>(pb.count) * pb.HW; break;
    case BNS_RULE_FEATURE: np.sampled_rows = static_cast<long>(pb.N) * pb.patch.ph * pb.patch.pw; break;
    default:
        np.sampled_rows = static_cast<long>(pb.count) * pb.HW;
        np.virt = plan_nhwc(pb.C, elem_bytes(sp->xv_dtype), np.sampled_rows, false);
        np.norm_virt = plan_nhwc(pb.C, elem_bytes(sp->xv_dtype), np.sampled_rows, false, true);
        break;
    }
    const int stat_eb = pb.rule == BNS_RULE_VIRTUAL ? elem_bytes(sp->xv_dtype) : eb;
    np.stat = plan_nhwc(pb.C, stat_eb, np.sampled_rows, pb.rule != BNS_RULE_FULL);
    np.direct = plan_nhwc_direct(pb.C, stat_eb, np.sampled_rows);
    // up to two batches of rows per thread: beyond that the chain of dependent batches inside the one block per
    // strip is longer than the extra launches it saves (256x512x28x28 with 2304 sampled rows measured 4-8 us slower
    // per layer; 256 rows 7-8 us faster, the CIFAR layers with 2048 rows 3 us faster)
    const long direct_rows = 2L * np.direct.shape.RL * kNhwcDirectUnroll;
    np.small_set = pb.rule != BNS_RULE_FULL && np.sampled_rows <= std::min<long>(g_direct_max, direct_rows);
    size_t off = kHeaderBytes;
    np.off_list = off;
    off += align_up(static_cast<size_t>(pb.N) * sizeof(int));
    np.off_stats = off;
    off += align_up(np.stat.partial_count() * sizeof(float4));
    np.off_bwd = off;
    off += align_up(np.main.partial_count() * sizeof(float2));
    np.off_bwd_v = off;
    if (pb.rule == BNS_RULE_VIRTUAL) off += align_up(np.virt.partial_count() * sizeof(float2));
    np.total = off;
    return BNS_OK;
}

// The sampled rows of the real tensor (or, for VIRTUAL, all rows of xv) as a RowSet.
RowSet nhwc_row_set(const NhwcProblem& np, const int* list) {
    const Problem& pb = np.pb;
    RowSet set{};
    set.total = static_cast<int>(np.sampled_rows);
    set.HW = pb.HW;
    set.H = pb.H;
    set.W = pb.W;
    set.list = list;
    set.begin = pb.begin;
    set.patch = pb.patch;
    set.mode = pb.rule == BNS_RULE_BATCH ? RowSet::kSamples : pb.rule == BNS_RULE_FEATURE ? RowSet::kPatches : RowSet::kAll;
    return set;
}

bns_status nhwc_stage_list(const NhwcProblem& np, const bns_sampling* sp, void* ws, cudaStream_t stream, const int** list) {
    *list = nullptr;
    if (np.pb.rule != BNS_RULE_BATCH || np.pb.contiguous) return BNS_OK;
    int* dev = ws_at<int>(ws, np.off_list);
    if (cudaMemcpyAsync(dev, sp->sample_idx, sizeof(int) * sp->k, cudaMemcpyHostToDevice, stream) != cudaSuccess)
        return BNS_ERR_CUDA;
    *list = dev;
    return BNS_OK;
}

#define BNS_NHWC_BY_TYPE_V(dtype, C_, CALL)                                  \
    do {                                                                     \
        const int V_ = nhwc_vector(C_, elem_bytes(dtype));                   \
        BNS_BY_TYPE_V(dtype, V_, CALL);                                      \
    } while (0)

template <typename... KArgs, typename... Args>
void launch_grid_block(int kind, void (*kernel)(KArgs...), dim3 grid, int threads, cudaStream_t s, Args&&... args) {
    LaunchScope scope(kind, s);
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = dim3(threads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = g_pdl ? 1 : 0;
    note_launch(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

template <typename... KArgs, typename... Args>
void launch_grid(int kind, void (*kernel)(KArgs...), dim3 grid, cudaStream_t s, Args&&... args) {
    launch_grid_block(kind, kernel, grid, kThreads, s, static_cast<Args&&>(args)...);
}

bns_status forward_nhwc_impl(const NhwcProblem& np, const bns_sampling* sp, const void* x, const float* gamma,
                             const float* beta, float eps, void* y, float* mean, float* invstd, void* ws,
                             cudaStream_t stream) {
    const Problem& pb = np.pb;
    unsigned* status;
    bns_status st = clear_status(pb, ws, stream, &status);
    if (st != BNS_OK) return st;
    const int* list = nullptr;
    st = nhwc_stage_list(np, sp, ws, stream, &list);
    if (st != BNS_OK) return st;
    const RowSet set = nhwc_row_set(np, list);
    const bool virt = pb.rule == BNS_RULE_VIRTUAL;
    const void* data = virt ? sp->xv : x;
    const int dt = virt ? sp->xv_dtype : pb.dtype;
    float4* partials = ws_at<float4>(ws, np.off_stats);
    if (np.small_set) {
        BNS_NHWC_BY_TYPE_V(dt, pb.C, (launch_grid(BNS_KERNEL_DIRECT_MOMENTS, nhwc_direct_moments_kernel<T, V>, np.direct.grid,
                                                  stream, in<T>(data), set, np.direct.shape, eps, mean, invstd, status)));
    } else {
        BNS_NHWC_BY_TYPE_V(dt, pb.C, (launch_grid(BNS_KERNEL_COL_MOMENTS, nhwc_moments_kernel<T, V>, np.stat.grid, stream,
                                                  in<T>(data), set, np.stat.shape, partials, status)));
        launch_grid_block(BNS_KERNEL_FINALIZE_STATS, nhwc_finalize_stats_kernel, dim3((pb.C + 31) / 32), kFinalizeThreads,
                          stream, static_cast<const float4*>(partials), static_cast<int>(np.stat.grid.x), pb.C,
                          static_cast<float>(1.0 / pb.s), eps, mean, invstd);
    }
    BNS_NHWC_BY_TYPE_V(pb.dtype, pb.C,
                       (launch_grid(BNS_KERNEL_NORMALIZE, nhwc_normalize_kernel<T, V>, np.norm.grid, stream, in<T>(x),
                                    out<T>(y), gamma, beta, mean, invstd, static_cast<int>(np.rows), np.norm.shape)));
    if (virt && sp->yv)
        BNS_NHWC_BY_TYPE_V(sp->xv_dtype, pb.C,
                           (launch_grid(BNS_KERNEL_NORMALIZE, nhwc_normalize_kernel<T, V>, np.norm_virt.grid, stream,
                                        in<T>(sp->xv), out<T>(sp->yv), gamma, beta, mean, invstd,
                                        static_cast<int>(np.sampled_rows), np.norm_virt.shape)));
    return last_error();
}

bns_status backward_nhwc_impl(const NhwcProblem& np, const bns_sampling* sp, const void* x, const void* dy,
                              const float* gamma, const float* mean, const float* invstd, void* dx, float* dgamma,
                              float* dbeta, void* ws, cudaStream_t stream) {
    const Problem& pb = np.pb;
    const bool full = pb.rule == BNS_RULE_FULL;
    const bool virt = pb.rule == BNS_RULE_VIRTUAL;
    float2* partials = ws_at<float2>(ws, np.off_bwd);
    float2* partials_v = (virt && sp->dyv) ? ws_at<float2>(ws, np.off_bwd_v) : nullptr;
    const int rows = static_cast<int>(np.rows);
    if (full)
        BNS_NHWC_BY_TYPE_V(pb.dtype, pb.C,
                           (launch_grid(BNS_KERNEL_BWD_REDUCE, nhwc_bwd_reduce_kernel<T, V, false>, np.main.grid, stream,
                                        in<T>(x), in<T>(dy), out<T>(nullptr), gamma, mean, invstd, rows, np.main.shape,
                                        partials)));
    else
        BNS_NHWC_BY_TYPE_V(pb.dtype, pb.C,
                           (launch_grid(BNS_KERNEL_BWD_REDUCE, nhwc_bwd_reduce_kernel<T, V, true>, np.main.grid, stream,
                                        in<T>(x), in<T>(dy), out<T>(dx), gamma, mean, invstd, rows, np.main.shape,
                                        partials)));
    if (partials_v)
        BNS_NHWC_BY_TYPE_V(sp->xv_dtype, pb.C,
                           (launch_grid(BNS_KERNEL_BWD_REDUCE, nhwc_bwd_reduce_kernel<T, V, false>, np.virt.grid, stream,
                                        in<T>(sp->xv), in<T>(sp->dyv), out<T>(nullptr), gamma, mean, invstd,
                                        static_cast<int>(np.sampled_rows), np.virt.shape, partials_v)));
    unsigned* status;
    bns_status st = clear_status(pb, ws, stream, &status);
    if (st != BNS_OK) return st;
    const int* list = nullptr;
    st = nhwc_stage_list(np, sp, ws, stream, &list);
    if (st != BNS_OK) return st;
    const RowSet set = nhwc_row_set(np, list);
    const float inv_s = static_cast<float>(1.0 / pb.s);
    if (np.small_set) {
        // one block per strip of channels combines the strip's sums and applies the statistics terms to its sampled set
        const void* src = virt ? sp->xv : x;
        const void* grad = virt ? sp->dyv : dy;
        void* dst = virt ? sp->dxv : dx;
        BNS_NHWC_BY_TYPE_V(virt ? sp->xv_dtype : pb.dtype, pb.C,
                           (launch_grid(BNS_KERNEL_DIRECT_FIXUP, nhwc_direct_finalize_fixup_kernel<T, V>, np.direct.grid,
                                        stream, in<T>(src), in<T>(grad), out<T>(dst), gamma, mean, invstd,
                                        static_cast<const float2*>(partials), static_cast<int>(np.main.grid.x),
                                        static_cast<const float2*>(partials_v), static_cast<int>(np.virt.grid.x), inv_s,
                                        set, np.direct.shape, dgamma, dbeta, status)));
        return last_error();
    }
    launch_grid_block(BNS_KERNEL_FINALIZE_BWD, nhwc_finalize_bwd_kernel, dim3((pb.C + 31) / 32), kFinalizeThreads, stream,
                      static_cast<const float2*>(partials), static_cast<int>(np.main.grid.x),
           static_cast<const float2*>(partials_v), static_cast<int>(np.virt.grid.x), pb.C, invstd, dgamma, dbeta);
    if (virt) {
        if (sp->dxv)
            BNS_NHWC_BY_TYPE_V(sp->xv_dtype, pb.C,
                               (launch_grid(BNS_KERNEL_COL_FIXUP, nhwc_fixup_kernel<T, V>, np.stat.grid, stream,
                                            in<T>(sp->xv), in<T>(sp->dyv), out<T>(sp->dxv), gamma, mean, invstd, dgamma,
                                            dbeta, inv_s, set, np.stat.shape, status)));
    } else {
        BNS_NHWC_BY_TYPE_V(pb.dtype, pb.C,
                           (launch_grid(BNS_KERNEL_COL_FIXUP, nhwc_fixup_kernel<T, V>, np.stat.grid, stream, in<T>(x),
                                        in<T>(dy), out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, set,
                                        np.stat.shape, status)));
    }
    return last_error();
}

bns_sampling full_rule() {
    bns_sampling sp;
    std::memset(&sp, 0, sizeof(sp));
    sp.rule = BNS_RULE_FULL;
    return sp;
}

}  // namespace

// Helper stream and events of bns_forward_backward_host, one set per device, created on first use and
// kept until the process ends (the only objects this library ever creates).  NULL if creation fails: the
// call then runs on the caller's stream alone.
constexpr int kHostChunks = 8;  // row chunks of the pipelined host-buffer call

struct CopyLane {
    cudaStream_t stream = nullptr;
    cudaEvent_t forward_done = nullptr, y_done = nullptr;
    cudaEvent_t chunk_done[2 * kHostChunks + 1] = {};  // forward chunks, backward chunks, the final fix-up
    bool tried = false;
};
CopyLane g_copy_lanes[64];
std::mutex g_copy_lanes_mutex;

CopyLane* copy_lane() {
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess || device < 0 || device >= 64) return nullptr;
    std::lock_guard<std::mutex> guard(g_copy_lanes_mutex);
    CopyLane& lane = g_copy_lanes[device];
    if (!lane.tried) {
        lane.tried = true;
        bool ok = cudaStreamCreateWithFlags(&lane.stream, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&lane.forward_done, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&lane.y_done, cudaEventDisableTiming) == cudaSuccess;
        for (cudaEvent_t& e : lane.chunk_done) ok = ok && cudaEventCreateWithFlags(&e, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            lane.stream = nullptr;
        }
    }
    return lane.stream ? &lane : nullptr;
}

// Device buffers of bns_forward_backward_host inside the caller's arena.
struct HostArena {
    void *d_x, *d_dy, *d_y, *d_dx, *ws;
    float *d_gamma, *d_beta, *d_mean, *d_invstd, *d_dgamma, *d_dbeta, *d_chunk_grads;
    size_t tensor_bytes, vector_bytes;
};

bool g_host_pipeline = true;  // overlap the two directions of the link by row chunks where the rule allows it

// The pipelined form of the host-buffer call.  Both directions of the link work at once for most of the
// call: what the statistics need goes up first (the sampled samples, or the patches of every map as one
// strided copy), then x goes up in row chunks while the normalised chunks of y already travel down; dy goes
// up in row chunks while backward pass 1 runs per chunk and the chunks of dx (correct everywhere but on the
// sampled set) travel down; last, the sums of the chunks are added, the sampled elements get their
// statistics terms, and only they are sent again.  One cudaMemcpyAsync (or cudaMemcpy3DAsync) per piece.
// Returns false, having enqueued nothing, when the rule or the shape does not allow it.
bool host_pipelined(const Problem& pb, const bns_sampling* sp, const void* x, const void* dy, const float* gamma,
                    const float* beta, float eps, void* y, void* dx, float* mean, float* invstd, float* dgamma,
                    float* dbeta, const HostArena& A, CopyLane* lane, cudaStream_t stream, bns_status* result) {
    const bool batch = pb.rule == BNS_RULE_BATCH && pb.contiguous;
    const bool feature = pb.rule == BNS_RULE_FEATURE && !pb.patch.offsets;
    if (!g_host_pipeline || !lane || !(batch || feature) || pb.N < 4 * kHostChunks) return false;
    const int eb = elem_bytes(pb.dtype);
    const size_t row_bytes = static_cast<size_t>(pb.P) * eb;
    auto at = [&](const void* p, int row) { return static_cast<const char*>(p) + static_cast<size_t>(row) * row_bytes; };
    auto at_mut = [&](void* p, int row) { return static_cast<char*>(p) + static_cast<size_t>(row) * row_bytes; };
    bool ok = true;
    // rows [r0, r0+rows) of a tensor over the link, leaving out the sampled samples of Batch Sampling (they
    // travel separately: up before everything else, down after the fix-up)
    auto copy_rows = [&](void* dst, const void* src, int r0, int rows, cudaMemcpyKind kind, cudaStream_t s) {
        const int skip_lo = batch ? pb.begin : 0, skip_hi = batch ? pb.begin + pb.count : 0;
        const int a0 = r0, a1 = std::min(r0 + rows, std::max(r0, skip_lo));      // before the sampled samples
        const int b0 = std::max(r0, std::min(r0 + rows, skip_hi)), b1 = r0 + rows;  // after them
        if (a1 > a0)
            ok &= cudaMemcpyAsync(at_mut(dst, a0), at(src, a0), (a1 - a0) * row_bytes, kind, s) == cudaSuccess;
        if (b1 > b0)
            ok &= cudaMemcpyAsync(at_mut(dst, b0), at(src, b0), (b1 - b0) * row_bytes, kind, s) == cudaSuccess;
    };
    auto copy_patches = [&](void* dst, const void* src, cudaMemcpyKind kind, cudaStream_t s) {
        cudaMemcpy3DParms p = {};
        const size_t pitch = static_cast<size_t>(pb.W) * eb;
        p.srcPtr = make_cudaPitchedPtr(const_cast<void*>(src), pitch, pitch, pb.H);
        p.dstPtr = make_cudaPitchedPtr(dst, pitch, pitch, pb.H);
        p.srcPos = p.dstPos = make_cudaPos(static_cast<size_t>(pb.patch.ow) * eb, pb.patch.oh, 0);
        p.extent = make_cudaExtent(static_cast<size_t>(pb.patch.pw) * eb, pb.patch.ph, static_cast<size_t>(pb.N) * pb.C);
        p.kind = kind;
        ok &= cudaMemcpy3DAsync(&p, s) == cudaSuccess;
    };
    ok &= cudaMemcpyAsync(A.d_gamma, gamma, A.vector_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(A.d_beta, beta, A.vector_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    // ---- forward: the sampled set first, statistics, then chunks up / normalise / chunks down
    if (batch)
        ok &= cudaMemcpyAsync(at_mut(A.d_x, pb.begin), at(x, pb.begin), pb.count * row_bytes, cudaMemcpyHostToDevice, stream) ==
              cudaSuccess;
    else
        copy_patches(A.d_x, x, cudaMemcpyHostToDevice, stream);
    if (!ok) {
        *result = BNS_ERR_CUDA;
        return true;
    }
    bns_status st = run_statistics(pb, sp, A.d_x, eps, A.d_mean, A.d_invstd, A.ws, stream);
    if (st != BNS_OK) {
        *result = st;
        return true;
    }
    for (int i = 0; i < kHostChunks; ++i) {
        const int r0 = static_cast<int>(static_cast<long long>(i) * pb.N / kHostChunks);
        const int rows = static_cast<int>(static_cast<long long>(i + 1) * pb.N / kHostChunks) - r0;
        copy_rows(A.d_x, x, r0, rows, cudaMemcpyHostToDevice, stream);
        const ColPlan pl = plan_col(pb.P, pb.HW, pb.C, rows, eb);
        BNS_BY_TYPE_V(pb.dtype, pl.V,
                      (launch_after_predecessor(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pl.grid(), stream,
                                                in<T>(at(A.d_x, r0)), out<T>(at_mut(A.d_y, r0)), A.d_gamma, A.d_beta, A.d_mean,
                                                A.d_invstd, RowOrder{RowOrder::kIdentity, rows, 0, 0}, pl.nchunks, pl.tiles,
                                                pb.HW, pb.P)));
        ok &= cudaEventRecord(lane->chunk_done[i], stream) == cudaSuccess;
        ok &= cudaStreamWaitEvent(lane->stream, lane->chunk_done[i], 0) == cudaSuccess;
        ok &= cudaMemcpyAsync(at_mut(y, r0), at(A.d_y, r0), rows * row_bytes, cudaMemcpyDeviceToHost, lane->stream) == cudaSuccess;
    }
    // ---- backward: chunks up / pass 1 per chunk / chunks of dx down
    for (int i = 0; i < kHostChunks; ++i) {
        const int r0 = static_cast<int>(static_cast<long long>(i) * pb.N / kHostChunks);
        const int rows = static_cast<int>(static_cast<long long>(i + 1) * pb.N / kHostChunks) - r0;
        ok &= cudaMemcpyAsync(at_mut(A.d_dy, r0), at(dy, r0), rows * row_bytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
        const ColPlan pl = plan_col(pb.P, pb.HW, pb.C, rows, eb);
        float* grads = A.d_chunk_grads + static_cast<size_t>(i) * 2 * pb.C;
        GradSink sink{ws_at<float2>(A.ws, pb.off_bwd), pl.layout(), nullptr, pl.layout(), A.d_invstd, grads, grads + pb.C};
        BNS_BY_TYPE_V(pb.dtype, pl.V,
                      (launch_after_predecessor(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, true>(pb.HW), pl.grid(), stream,
                                                in<T>(at(A.d_x, r0)), in<T>(at(A.d_dy, r0)), out<T>(at_mut(A.d_dx, r0)), A.d_gamma,
                                                A.d_mean, A.d_invstd, RowOrder{RowOrder::kIdentity, rows, 0, 0}, pl.nchunks,
                                                pl.tiles, pb.HW, pb.P, false, sink)));
        launch(BNS_KERNEL_FINALIZE_BWD, finalize_bwd_kernel, warp_per_channel_grid(pb.C), stream, sink, pb.C, pb.HW);
        ok &= cudaEventRecord(lane->chunk_done[kHostChunks + i], stream) == cudaSuccess;
        ok &= cudaStreamWaitEvent(lane->stream, lane->chunk_done[kHostChunks + i], 0) == cudaSuccess;
        copy_rows(dx, A.d_dx, r0, rows, cudaMemcpyDeviceToHost, lane->stream);
    }
    // ---- the sums of all chunks, the statistics terms on the sampled set, and that set once more down the link
    launch(BNS_KERNEL_VECTOR, sum_chunk_grads_kernel, per_channel_grid(pb.C), stream,
           static_cast<const float*>(A.d_chunk_grads), kHostChunks, pb.C, A.d_dgamma, A.d_dbeta);
    const float inv_s = static_cast<float>(1.0 / pb.s);
    if (batch) {
        const ColPlan& pv = pb.stat_plan;
        BNS_BY_TYPE_V(pb.dtype, pv.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pv.grid(), stream, in<T>(A.d_x), in<T>(A.d_dy),
                              out<T>(A.d_dx), A.d_gamma, A.d_mean, A.d_invstd, A.d_dgamma, A.d_dbeta, inv_s,
                              static_cast<const int*>(nullptr), pb.begin, RowOrder{RowOrder::kIdentity, pv.rows, 0, 0},
                              pv.nchunks, pv.tiles, pb.HW, pb.P, GradSink{}, 0)));
    } else {
        const PatchPlan& pp = pb.patch_plan;
        BNS_BY_TYPE(pb.dtype, (launch(BNS_KERNEL_PATCH_FIXUP, patch_fixup_kernel<T>, pp.grid(), stream, in<T>(A.d_x),
                                      in<T>(A.d_dy), out<T>(A.d_dx), A.d_gamma, A.d_mean, A.d_invstd, A.d_dgamma, A.d_dbeta,
                                      inv_s, pb.patch, pb.N, pb.C, pb.H, pb.W, pp.nchunks, pp.tiles,
                                      static_cast<unsigned*>(nullptr), GradSink{}, 0)));
    }
    ok &= cudaEventRecord(lane->chunk_done[2 * kHostChunks], stream) == cudaSuccess;
    ok &= cudaStreamWaitEvent(lane->stream, lane->chunk_done[2 * kHostChunks], 0) == cudaSuccess;
    if (batch)
        ok &= cudaMemcpyAsync(at_mut(dx, pb.begin), at(A.d_dx, pb.begin), pb.count * row_bytes, cudaMemcpyDeviceToHost,
                              lane->stream) == cudaSuccess;
    else
        copy_patches(dx, A.d_dx, cudaMemcpyDeviceToHost, lane->stream);
    ok &= cudaEventRecord(lane->y_done, lane->stream) == cudaSuccess;
    ok &= cudaStreamWaitEvent(stream, lane->y_done, 0) == cudaSuccess;  // the helper joins the caller's stream
    ok &= cudaMemcpyAsync(mean, A.d_mean, A.vector_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(invstd, A.d_invstd, A.vector_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(dgamma, A.d_dgamma, A.vector_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(dbeta, A.d_dbeta, A.vector_bytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    const bns_status launches = last_error();
    *result = !ok ? BNS_ERR_CUDA : launches;
    return true;
}

// ======================================================================================== C ABI
extern "C" {

size_t bns_workspace_bytes(const bns_shape* shape, const bns_sampling* sampling) {
    Problem pb;
    if (make_problem(shape, sampling, pb) != BNS_OK) return 0;
    return pb.total;
}

bns_status bns_forward(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps,
                       const bns_sampling* sampling, void* y, float* mean, float* invstd, void* workspace,
                       size_t workspace_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !y || !mean || !invstd) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    return forward_impl(pb, sampling, x, gamma, beta, eps, y, mean, invstd, workspace,
                        static_cast<cudaStream_t>(cuda_stream));
}

bns_status bns_backward(const bns_shape* shape, const void* x, const void* dy, const float* gamma, const float* mean,
                        const float* invstd, const bns_sampling* sampling, void* dx, float* dgamma, float* dbeta,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !dy || !gamma || !mean || !invstd || !dx || !dgamma || !dbeta) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    return backward_impl(pb, sampling, x, dy, gamma, mean, invstd, dx, dgamma, dbeta, workspace,
                         static_cast<cudaStream_t>(cuda_stream));
}

bns_status bns_full_bn(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps, void* y,
                       float* mean, float* invstd, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    bns_sampling sp = full_rule();
    return bns_forward(shape, x, gamma, beta, eps, &sp, y, mean, invstd, workspace, workspace_bytes, cuda_stream);
}

size_t bns_host_arena_bytes(const bns_shape* shape, const bns_sampling* sampling) {
    Problem pb;
    if (make_problem(shape, sampling, pb) != BNS_OK) return 0;
    const size_t tensor = align_up(pb.elems * elem_bytes(pb.dtype));
    const size_t vec = align_up(static_cast<size_t>(pb.C) * sizeof(float));
    return 4 * tensor + 6 * vec + align_up(pb.total) + 2 * kHostChunks * vec;
}

bns_status bns_forward_backward_host(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                                     const float* beta, float eps, const bns_sampling* sampling, void* y, void* dx,
                                     float* mean, float* invstd, float* dgamma, float* dbeta, void* arena,
                                     size_t arena_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !dy || !gamma || !beta || !y || !dx || !mean || !invstd || !dgamma || !dbeta) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    const size_t need = bns_host_arena_bytes(shape, sampling);
    if (!arena || (reinterpret_cast<uintptr_t>(arena) & (kAlign - 1)) || arena_bytes < need) return BNS_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t tbytes = pb.elems * elem_bytes(pb.dtype);
    const size_t tensor = align_up(tbytes);
    const size_t vbytes = static_cast<size_t>(pb.C) * sizeof(float);
    const size_t vec = align_up(vbytes);
    char* base = static_cast<char*>(arena);
    void* d_x = base;
    void* d_dy = base + tensor;
    void* d_y = base + 2 * tensor;
    void* d_dx = base + 3 * tensor;
    float* d_vec[6];
    for (int i = 0; i < 6; ++i) d_vec[i] = reinterpret_cast<float*>(base + 4 * tensor + i * vec);
    void* ws = base + 4 * tensor + 6 * vec;
    float *d_gamma = d_vec[0], *d_beta = d_vec[1], *d_mean = d_vec[2], *d_invstd = d_vec[3], *d_dgamma = d_vec[4],
          *d_dbeta = d_vec[5];
    {
        void* after_ws = base + 4 * tensor + 6 * vec + align_up(pb.total);
        const HostArena A{d_x, d_dy, d_y, d_dx, ws, d_gamma, d_beta, d_mean, d_invstd, d_dgamma, d_dbeta,
                          static_cast<float*>(after_ws), tbytes, vbytes};
        bns_status piped = BNS_OK;
        if (host_pipelined(pb, sampling, x, dy, gamma, beta, eps, y, dx, mean, invstd, dgamma, dbeta, A, copy_lane(), stream,
                           &piped))
            return piped;
    }
    bool ok = true;
    ok &= cudaMemcpyAsync(d_x, x, tbytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_gamma, gamma, vbytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(d_beta, beta, vbytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) return BNS_ERR_CUDA;
    st = forward_impl(pb, sampling, d_x, d_gamma, d_beta, eps, d_y, d_mean, d_invstd, ws, stream);
    if (st != BNS_OK) return st;
    // y travels to the host on a helper stream while dy travels to the device on the caller's: the two
    // directions of the link are independent.  The helper joins the caller's stream again at the end.
    CopyLane* lane = copy_lane();
    if (lane) {
        ok &= cudaEventRecord(lane->forward_done, stream) == cudaSuccess;
        ok &= cudaStreamWaitEvent(lane->stream, lane->forward_done, 0) == cudaSuccess;
        ok &= cudaMemcpyAsync(y, d_y, tbytes, cudaMemcpyDeviceToHost, lane->stream) == cudaSuccess;
        ok &= cudaEventRecord(lane->y_done, lane->stream) == cudaSuccess;
    } else {
        ok &= cudaMemcpyAsync(y, d_y, tbytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    }
    ok &= cudaMemcpyAsync(d_dy, dy, tbytes, cudaMemcpyHostToDevice, stream) == cudaSuccess;
    if (!ok) return BNS_ERR_CUDA;
    st = backward_impl(pb, sampling, d_x, d_dy, d_gamma, d_mean, d_invstd, d_dx, d_dgamma, d_dbeta, ws, stream);
    if (st != BNS_OK) return st;
    if (lane) ok &= cudaStreamWaitEvent(stream, lane->y_done, 0) == cudaSuccess;
    ok &= cudaMemcpyAsync(dx, d_dx, tbytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(mean, d_mean, vbytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(invstd, d_invstd, vbytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(dgamma, d_dgamma, vbytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    ok &= cudaMemcpyAsync(dbeta, d_dbeta, vbytes, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
    return ok ? BNS_OK : BNS_ERR_CUDA;
}

bns_status bns_debug_selection_mask(const bns_shape* shape, const bns_sampling* sampling, uint8_t* mask,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!mask) return BNS_ERR_NULL;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int* list = nullptr;
    st = stage_list(pb, sampling, workspace, stream, &list);
    if (st != BNS_OK) return st;
    unsigned* status;
    st = clear_status(pb, workspace, stream, &status);
    if (st != BNS_OK) return st;
    const size_t blocks = std::min<size_t>((pb.elems + kThreads - 1) / kThreads, static_cast<size_t>(sm_count()) * 32);
    launch_after_predecessor(BNS_KERNEL_MASK, selection_mask_kernel, static_cast<unsigned>(blocks), stream, mask, pb.rule,
                             list, pb.begin, pb.count, pb.patch, pb.N, pb.C, pb.H, pb.W, status);
    return last_error();
}

bns_status bns_workspace_status(const void* workspace, uint32_t* flags, void* cuda_stream) {
    if (!workspace || !flags) return BNS_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(flags, workspace, sizeof(uint32_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return BNS_ERR_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? BNS_OK : BNS_ERR_CUDA;
}

const char* bns_status_string(bns_status status) {
    switch (status) {
    case BNS_OK: return "ok";
    case BNS_ERR_NULL: return "a required pointer is NULL";
    case BNS_ERR_SHAPE: return "invalid shape or eps";
    case BNS_ERR_RULE: return "invalid sampling rule";
    case BNS_ERR_INDEX: return "sample index or patch offset out of range or repeated";
    case BNS_ERR_DTYPE: return "unknown element type";
    case BNS_ERR_ALIGN: return "pointer not sufficiently aligned";
    case BNS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case BNS_ERR_CUDA: return "CUDA runtime error";
    }
    return "unknown status";
}

uint64_t bns_launch_count(void) { return g_launches.load(); }
void bns_launch_count_reset(void) { g_launches.store(0); }

void bns_profile_enable(int on) {
    for (TimedLaunch& t : g_timed) {
        g_free_events.push_back(t.start);
        g_free_events.push_back(t.stop);
    }
    g_timed.clear();
    g_profile = on != 0;
}

bns_status bns_profile_read(int kernel_kind, int* launches, float* total_ms) {
    if (!launches || !total_ms) return BNS_ERR_NULL;
    *launches = 0;
    *total_ms = 0.f;
    for (const TimedLaunch& t : g_timed) {
        if (t.kind != kernel_kind) continue;
        if (cudaEventSynchronize(t.stop) != cudaSuccess) return BNS_ERR_CUDA;
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, t.start, t.stop) != cudaSuccess) return BNS_ERR_CUDA;
        *launches += 1;
        *total_ms += ms;
    }
    return BNS_OK;
}

int bns_set_tuning(const char* name, int value) {
    if (!name) return BNS_ERR_NULL;
    struct Knob {
        const char* name;
        int* ivalue;
        bool* bvalue;
        bool zero_allowed;  // 0 has a meaning of its own for this knob (automatic, or never)
    } knobs[] = {{"target_blocks", &g_target_blocks, nullptr, true},
                 {"min_chunk", &g_min_chunk, nullptr, false},
                 {"full_min_chunk", &g_full_min_chunk, nullptr, false},
                 {"stat_target_blocks", &g_stat_target_blocks, nullptr, true},
                 {"stat_min_chunk", &g_stat_min_chunk, nullptr, false},
                 {"direct_max", &g_direct_max, nullptr, true},
                 {"nhwc_blocks", &g_nhwc_blocks, nullptr, true},
                 {"slab", nullptr, &g_slab, false},
                 {"slab_small_sets", nullptr, &g_slab_small_sets, false},
                 {"slab_cta_kb", &g_slab_cta_kb, nullptr, false},
                 {"slab_min_ctas", &g_slab_min_ctas, nullptr, true},
                 {"slab_max_mb", &g_slab_max_mb, nullptr, false},
                 {"slab_cluster_max", &g_slab_cluster_max, nullptr, false},
                 {"per_channel_min_hw", &g_per_channel_min_hw, nullptr, false},
                 {"fold_finalize", nullptr, &g_fold_finalize, false},
                 {"host_pipeline", nullptr, &g_host_pipeline, false},
                 {"pdl", nullptr, &g_pdl, false},
                 {"l2_order", nullptr, &g_l2_order, false}};
    for (const Knob& k : knobs) {
        if (std::strcmp(name, k.name) != 0) continue;
        if (k.ivalue) {
            if (value < (k.zero_allowed ? 0 : 1)) return BNS_ERR_SHAPE;
            if (k.ivalue == &g_slab_cluster_max && value > 8) return BNS_ERR_SHAPE;  // 8 is the portable cluster limit
            *k.ivalue = value;
        } else {
            *k.bvalue = value != 0;
        }
        return BNS_OK;
    }
    return BNS_ERR_RULE;
}

int bns_slab_plan(const bns_shape* shape, const bns_sampling* sampling, int backward, int32_t* plan) {
    Problem pb;
    if (!plan) return 0;
    if (make_problem(shape, sampling, pb) != BNS_OK) return 0;
    const SlabPlan& pl = backward ? pb.slab_bwd : pb.slab_fwd;
    if (!pl.ok) return 0;
    plan[0] = pl.geo.G;
    plan[1] = pl.geo.R;
    plan[2] = pl.geo.rows_max;
    plan[3] = static_cast<int32_t>(pl.geo.total_bytes);
    plan[4] = static_cast<int32_t>(pl.grid);
    plan[5] = pl.geo.RL;
    return 1;
}

bns_status bns_wait_timeouts(uint32_t* count, void* cuda_stream) {
    if (!count) return BNS_ERR_NULL;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyFromSymbolAsync(count, g_wait_timeouts, sizeof(uint32_t), 0, cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return BNS_ERR_CUDA;
    return cudaStreamSynchronize(stream) == cudaSuccess ? BNS_OK : BNS_ERR_CUDA;
}

const char* bns_kernel_name(int kernel_kind) {
    switch (kernel_kind) {
    case BNS_KERNEL_COL_MOMENTS: return "col_moments_kernel";
    case BNS_KERNEL_PATCH_MOMENTS: return "patch_moments_kernel";
    case BNS_KERNEL_FINALIZE_STATS: return "finalize_stats_kernel";
    case BNS_KERNEL_NORMALIZE: return "col_normalize_kernel";
    case BNS_KERNEL_BWD_REDUCE: return "col_bwd_reduce_kernel";
    case BNS_KERNEL_FINALIZE_BWD: return "finalize_bwd_kernel";
    case BNS_KERNEL_COL_FIXUP: return "col_fixup_kernel";
    case BNS_KERNEL_PATCH_FIXUP: return "patch_fixup_kernel";
    case BNS_KERNEL_MASK: return "selection_mask_kernel";
    case BNS_KERNEL_DIRECT_MOMENTS: return "direct_moments_kernel";
    case BNS_KERNEL_DIRECT_FIXUP: return "direct_finalize_fixup_kernel";
    case BNS_KERNEL_VECTOR: return "per-channel vector kernels";
    case BNS_KERNEL_SLAB_FORWARD: return "slab_forward_kernel";
    case BNS_KERNEL_SLAB_BACKWARD: return "slab_backward_kernel";
    }
    return "unknown";
}

// ---------------------------------------------------------------------------------------- Eq. 4 and Appendix D
size_t bns_workspace_bytes_mixed(const bns_shape* shape, const bns_sampling* sampling) {
    MixedProblem mp;
    if (make_mixed(shape, sampling, 0.5f, mp) != BNS_OK) return 0;
    return mp.total;
}

bns_status bns_forward_mixed(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps,
                             float mix, const bns_sampling* sampling, void* y, float* mean, float* invstd, float* mean_s,
                             float* mean_v, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    MixedProblem mp;
    bns_status st = make_mixed(shape, sampling, mix, mp);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !y || !mean || !invstd || !mean_s || !mean_v) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) || workspace_bytes < mp.total)
        return BNS_ERR_WORKSPACE;
    return forward_mixed_impl(mp, sampling, x, gamma, beta, eps, mix, y, mean, invstd, mean_s, mean_v, workspace,
                              static_cast<cudaStream_t>(cuda_stream));
}

bns_status bns_backward_mixed(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                              const float* mean, const float* invstd, const float* mean_s, const float* mean_v, float mix,
                              const bns_sampling* sampling, void* dx, float* dgamma, float* dbeta, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
    MixedProblem mp;
    bns_status st = make_mixed(shape, sampling, mix, mp);
    if (st != BNS_OK) return st;
    if (!x || !dy || !gamma || !mean || !invstd || !mean_s || !mean_v || !dx || !dgamma || !dbeta) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx)) return BNS_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) || workspace_bytes < mp.total)
        return BNS_ERR_WORKSPACE;
    return backward_mixed_impl(mp, sampling, x, dy, gamma, mean, invstd, mean_s, mean_v, mix, dx, dgamma, dbeta, workspace,
                               static_cast<cudaStream_t>(cuda_stream));
}

bns_status bns_update_moving_average(int C, const float* mean, const float* invstd, float eps, float alpha,
                                     int first_iteration, float* mean_ma, float* var_ma, void* cuda_stream) {
    if (C <= 0 || !(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!(alpha >= 0.f && alpha <= 1.f)) return BNS_ERR_RULE;
    if (!mean || !invstd || !mean_ma || !var_ma) return BNS_ERR_NULL;
    launch(BNS_KERNEL_VECTOR, moving_average_kernel, per_channel_grid(C), static_cast<cudaStream_t>(cuda_stream), mean,
           invstd, eps, alpha, first_iteration ? 1 : 0, C, mean_ma, var_ma);
    return last_error();
}

bns_status bns_forward_training(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps,
                                const bns_sampling* sampling, float alpha, int first_iteration, float* mean_ma,
                                float* var_ma, void* y, float* mean, float* invstd, void* workspace,
                                size_t workspace_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !y || !mean || !invstd || !mean_ma || !var_ma) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!(alpha >= 0.f && alpha <= 1.f)) return BNS_ERR_RULE;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    const MovingAverage ma{alpha, first_iteration ? 1 : 0, mean_ma, var_ma};
    return forward_impl(pb, sampling, x, gamma, beta, eps, y, mean, invstd, workspace,
                        static_cast<cudaStream_t>(cuda_stream), ma);
}

bns_status bns_inference_forward(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps,
                                 const float* mean_ma, const float* var_ma, void* y, void* workspace,
                                 size_t workspace_bytes, void* cuda_stream) {
    bns_sampling sp = full_rule();
    Problem pb;
    bns_status st = make_problem(shape, &sp, pb);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !mean_ma || !var_ma || !y) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    if (pb.total - pb.off_stats < static_cast<size_t>(pb.C) * sizeof(float)) return BNS_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    float* invstd = ws_at<float>(workspace, pb.off_stats);
    launch(BNS_KERNEL_VECTOR, invstd_from_var_kernel, per_channel_grid(pb.C), stream, var_ma, eps, pb.C, invstd);
    const ColPlan& pl = pb.main_plan;
    BNS_BY_TYPE_V(pb.dtype, pl.V,
                  (launch(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pl.grid(), stream, in<T>(x), out<T>(y), gamma,
                          beta, mean_ma, invstd, RowOrder{RowOrder::kIdentity, pb.N, 0, 0}, pl.nchunks, pl.tiles, pb.HW,
                          pb.P)));
    return last_error();
}

// ---------------------------------------------------------------------------------------- statistics shared by several GPUs
bns_status bns_sync_local_moments(const bns_shape* shape, const void* x, const bns_sampling* sampling, float eps,
                                  float* moments, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (!sampling) {
        // this rank samples nothing: a count of zero, which the merge passes over
        bns_status sc = check_shape(shape);
        if (sc != BNS_OK) return sc;
        if (!moments) return BNS_ERR_NULL;
        return cudaMemsetAsync(moments, 0, 3 * static_cast<size_t>(shape->C) * sizeof(float),
                               static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess
                   ? BNS_OK
                   : BNS_ERR_CUDA;
    }
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !moments) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = run_statistics(pb, sampling, x, eps, moments + pb.C, moments + 2 * pb.C, workspace, stream);
    if (st != BNS_OK) return st;
    launch(BNS_KERNEL_VECTOR, moments_rows_kernel, per_channel_grid(pb.C), stream, moments, static_cast<float>(pb.s), eps,
           pb.C);
    return last_error();
}

bns_status bns_sync_merge_moments(int C, int ranks, const float* moments, float eps, float* mean, float* invstd,
                                  float* count, void* cuda_stream) {
    if (C <= 0 || ranks <= 0 || !(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!moments || !mean || !invstd) return BNS_ERR_NULL;
    launch(BNS_KERNEL_VECTOR, merge_rank_moments_kernel, per_channel_grid(C), static_cast<cudaStream_t>(cuda_stream),
           moments, ranks, C, eps, mean, invstd, count);
    return last_error();
}

bns_status bns_sync_normalize(const bns_shape* shape, const void* x, const float* gamma, const float* beta,
                              const float* mean, const float* invstd, void* y, void* cuda_stream) {
    bns_sampling sp = full_rule();
    Problem pb;
    bns_status st = make_problem(shape, &sp, pb);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !mean || !invstd || !y) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    const ColPlan& pl = pb.main_plan;
    BNS_BY_TYPE_V(pb.dtype, pl.V,
                  (launch_after_predecessor(BNS_KERNEL_NORMALIZE, col_normalize_kernel<T, V>, pl.grid(),
                                            static_cast<cudaStream_t>(cuda_stream), in<T>(x), out<T>(y), gamma, beta, mean,
                                            invstd, RowOrder{RowOrder::kIdentity, pb.N, 0, 0},
                          pl.nchunks, pl.tiles, pb.HW, pb.P)));
    return last_error();
}

bns_status bns_sync_backward_sums(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                                  const float* mean, const float* invstd, const bns_sampling* virtual_rows, void* dx,
                                  float* sums, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    bns_sampling full = full_rule();
    if (virtual_rows && virtual_rows->rule != BNS_RULE_VIRTUAL) return BNS_ERR_RULE;
    const bool with_virtual = virtual_rows && virtual_rows->dyv;
    Problem pb;
    bns_status st = make_problem(shape, with_virtual ? virtual_rows : &full, pb);
    if (st != BNS_OK) return st;
    if (!x || !dy || !gamma || !mean || !invstd || !dx || !sums) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const ColPlan& pl = pb.main_plan;
    const ColPlan& pv = pb.stat_plan;
    // row 0: sum dy (dbeta), row 1: sum dy xhat (dgamma) over this rank's elements (and its virtual rows)
    GradSink sink{ws_at<float2>(workspace, pb.off_bwd), pl.layout(),
                  with_virtual ? ws_at<float2>(workspace, pb.off_bwd_v) : nullptr, pv.layout(), invstd, sums + pb.C, sums};
    BNS_BY_TYPE_V(pb.dtype, pl.V,
                  (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, true>(pb.HW), pl.grid(), stream, in<T>(x), in<T>(dy),
                          out<T>(dx), gamma, mean, invstd, RowOrder{RowOrder::kIdentity, pb.N, 0, 0}, pl.nchunks, pl.tiles,
                          pb.HW, pb.P, false, sink)));
    if (with_virtual)
        BNS_BY_TYPE_V(virtual_rows->xv_dtype, pv.V,
                      (launch(BNS_KERNEL_BWD_REDUCE, bwd_reduce_variant<T, V, false>(pb.HW), pv.grid(), stream,
                              in<T>(virtual_rows->xv), in<T>(virtual_rows->dyv), out<T>(nullptr), gamma, mean, invstd,
                              RowOrder{RowOrder::kIdentity, pv.rows, 0, 0}, pv.nchunks, pv.tiles, pb.HW, pb.P, true, sink)));
    launch(BNS_KERNEL_FINALIZE_BWD, finalize_bwd_kernel, warp_per_channel_grid(pb.C), stream, sink, pb.C, pb.HW);
    return last_error();
}

bns_status bns_sync_backward_apply(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                                   const float* mean, const float* invstd, const bns_sampling* sampling,
                                   const float* sums, const float* count, void* dx, void* workspace,
                                   size_t workspace_bytes, void* cuda_stream) {
    if (!sampling) return check_shape(shape);  // nothing of this rank is in the sampled set: dx stays as it is
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !dy || !gamma || !mean || !invstd || !sums || !count || !dx) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    if (pb.total - pb.off_stats < 2 * static_cast<size_t>(pb.C) * sizeof(float)) return BNS_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the summed rows divided by the sampled count of all ranks, which stays on the device: the fix-up
    // kernels then run with 1/s = 1
    float* shares = ws_at<float>(workspace, pb.off_stats);
    launch(BNS_KERNEL_VECTOR, per_point_shares_kernel, per_channel_grid(pb.C), stream, sums, count, pb.C, shares);
    const float* dbeta = shares;
    const float* dgamma = shares + pb.C;
    const float inv_s = 1.0f;
    const ColPlan& pl = pb.main_plan;
    const ColPlan& pv = pb.stat_plan;
    if (pb.rule == BNS_RULE_FULL) {
        BNS_BY_TYPE_V(pb.dtype, pl.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pl.grid(), stream, in<T>(x), in<T>(dy),
                              out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, static_cast<const int*>(nullptr), 0,
                              RowOrder{RowOrder::kIdentity, pl.rows, 0, 0}, pl.nchunks, pl.tiles, pb.HW, pb.P, GradSink{}, 0)));
    } else if (pb.rule == BNS_RULE_BATCH) {
        const int* list = nullptr;
        st = stage_list(pb, sampling, workspace, stream, &list);
        if (st != BNS_OK) return st;
        BNS_BY_TYPE_V(pb.dtype, pv.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pv.grid(), stream, in<T>(x), in<T>(dy),
                              out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, list, pb.begin,
                              RowOrder{RowOrder::kIdentity, pv.rows, 0, 0}, pv.nchunks, pv.tiles, pb.HW, pb.P, GradSink{}, 0)));
    } else if (pb.rule == BNS_RULE_FEATURE) {
        unsigned* status;
        st = clear_status(pb, workspace, stream, &status);
        if (st != BNS_OK) return st;
        const PatchPlan& pp = pb.patch_plan;
        BNS_BY_TYPE(pb.dtype, (launch(BNS_KERNEL_PATCH_FIXUP, patch_fixup_kernel<T>, pp.grid(), stream, in<T>(x), in<T>(dy),
                                      out<T>(dx), gamma, mean, invstd, dgamma, dbeta, inv_s, pb.patch, pb.N, pb.C, pb.H,
                                      pb.W, pp.nchunks, pp.tiles, status, GradSink{}, 0)));
    } else if (sampling->dxv) {
        // the virtual samples that this rank fed into the statistics: every one of them takes the upper branch
        BNS_BY_TYPE_V(sampling->xv_dtype, pv.V,
                      (launch(BNS_KERNEL_COL_FIXUP, col_fixup_kernel<T, V>, pv.grid(), stream, in<T>(sampling->xv),
                              in<T>(sampling->dyv), out<T>(sampling->dxv), gamma, mean, invstd, dgamma, dbeta, inv_s,
                              static_cast<const int*>(nullptr), 0, RowOrder{RowOrder::kIdentity, pv.rows, 0, 0}, pv.nchunks,
                              pv.tiles, pb.HW, pb.P, GradSink{}, 0)));
    }
    return last_error();
}

// ---------------------------------------------------------------------------------------- BN + residual add + ReLU
bns_status bns_forward_relu(const bns_shape* shape, const void* x, const void* residual, const float* gamma,
                            const float* beta, float eps, const bns_sampling* sampling, void* y, float* mean,
                            float* invstd, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (pb.rule == BNS_RULE_VIRTUAL) return BNS_ERR_RULE;
    if (!x || !gamma || !beta || !y || !mean || !invstd) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y) || !aligned16(residual)) return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = run_statistics(pb, sampling, x, eps, mean, invstd, workspace, stream);
    if (st != BNS_OK) return st;
    const ColPlan& pl = pb.main_plan;
    BNS_BY_TYPE_V(pb.dtype, pl.V,
                  (launch(BNS_KERNEL_NORMALIZE, act_normalize_kernel<T, V>, pl.grid(), stream, in<T>(x), in<T>(residual),
                          out<T>(y), gamma, beta, mean, invstd, RowOrder{RowOrder::kIdentity, pl.rows, 0, 0}, pl.nchunks,
                          pl.tiles, pb.HW, pb.P)));
    return last_error();
}

bns_status bns_backward_relu(const bns_shape* shape, const void* x, const void* residual, const void* dy,
                             const float* gamma, const float* beta, const float* mean, const float* invstd,
                             const bns_sampling* sampling, void* dx, void* dresidual, float* dgamma, float* dbeta,
                             void* workspace, size_t workspace_bytes, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (pb.rule == BNS_RULE_VIRTUAL) return BNS_ERR_RULE;
    if (!x || !dy || !gamma || !beta || !mean || !invstd || !dx || !dgamma || !dbeta) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx) || !aligned16(residual) || !aligned16(dresidual))
        return BNS_ERR_ALIGN;
    st = check_workspace(pb, workspace, workspace_bytes);
    if (st != BNS_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const ColPlan& pl = pb.main_plan;
    const ColPlan& pv = pb.stat_plan;
    GradSink sink{ws_at<float2>(workspace, pb.off_bwd), pl.layout(), nullptr, pl.layout(), invstd, dgamma, dbeta};
    BNS_BY_TYPE_V(pb.dtype, pl.V,
                  (launch(BNS_KERNEL_BWD_REDUCE, act_bwd_reduce_kernel<T, V>, pl.grid(), stream, in<T>(x), in<T>(residual),
                          in<T>(dy), out<T>(dx), out<T>(dresidual), gamma, beta, mean, invstd,
                          RowOrder{RowOrder::kIdentity, pl.rows, 0, 0}, pl.nchunks, pl.tiles, pb.HW, pb.P, sink)));
    // the second pass finishes the sums of Eq. 5 itself where its tiles meet few channels (as in backward_impl)
    const int second_pass_slots = pb.rule == BNS_RULE_FEATURE ? pb.patch_plan.max_slots
                                  : pb.rule == BNS_RULE_FULL  ? pl.max_slots
                                                              : pv.max_slots;
    const int fold = g_fold_finalize && pb.rule != BNS_RULE_FULL && second_pass_slots <= kFoldSlots ? 1 : 0;
    if (!fold) launch(BNS_KERNEL_FINALIZE_BWD, finalize_bwd_kernel, warp_per_channel_grid(pb.C), stream, sink, pb.C, pb.HW);
    const float inv_s = static_cast<float>(1.0 / pb.s);
    if (pb.rule == BNS_RULE_FEATURE) {
        unsigned* status;
        st = clear_status(pb, workspace, stream, &status);
        if (st != BNS_OK) return st;
        const PatchPlan& pp = pb.patch_plan;
        BNS_BY_TYPE(pb.dtype, (launch(BNS_KERNEL_PATCH_FIXUP, act_patch_fixup_kernel<T>, pp.grid(), stream, in<T>(x),
                                      in<T>(residual), in<T>(dy), out<T>(dx), gamma, beta, mean, invstd, dgamma, dbeta,
                                      inv_s, pb.patch, pb.N, pb.C, pb.H, pb.W, pp.nchunks, pp.tiles, status, sink,
                                      fold)));
    } else {
        const int* list = nullptr;
        st = stage_list(pb, sampling, workspace, stream, &list);
        if (st != BNS_OK) return st;
        const ColPlan& pf = pb.rule == BNS_RULE_FULL ? pl : pv;
        BNS_BY_TYPE_V(pb.dtype, pf.V,
                      (launch(BNS_KERNEL_COL_FIXUP, act_col_fixup_kernel<T, V>, pf.grid(), stream, in<T>(x),
                              in<T>(residual), in<T>(dy), out<T>(dx), gamma, beta, mean, invstd, dgamma, dbeta, inv_s,
                              list, pb.rule == BNS_RULE_BATCH ? pb.begin : 0,
                              RowOrder{RowOrder::kIdentity, pf.rows, 0, 0}, pf.nchunks, pf.tiles, pb.HW, pb.P, sink, fold)));
    }
    return last_error();
}

// ---------------------------------------------------------------------------------------- channels-last (NHWC)
size_t bns_workspace_bytes_nhwc(const bns_shape* shape, const bns_sampling* sampling) {
    NhwcProblem np;
    if (make_nhwc(shape, sampling, np) != BNS_OK) return 0;
    return np.total;
}

bns_status bns_forward_nhwc(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps,
                            const bns_sampling* sampling, void* y, float* mean, float* invstd, void* workspace,
                            size_t workspace_bytes, void* cuda_stream) {
    NhwcProblem np;
    bns_status st = make_nhwc(shape, sampling, np);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !y || !mean || !invstd) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) || workspace_bytes < np.total)
        return BNS_ERR_WORKSPACE;
    return forward_nhwc_impl(np, sampling, x, gamma, beta, eps, y, mean, invstd, workspace,
                             static_cast<cudaStream_t>(cuda_stream));
}

bns_status bns_backward_nhwc(const bns_shape* shape, const void* x, const void* dy, const float* gamma,
                             const float* mean, const float* invstd, const bns_sampling* sampling, void* dx,
                             float* dgamma, float* dbeta, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    NhwcProblem np;
    bns_status st = make_nhwc(shape, sampling, np);
    if (st != BNS_OK) return st;
    if (!x || !dy || !gamma || !mean || !invstd || !dx || !dgamma || !dbeta) return BNS_ERR_NULL;
    if (!aligned16(x) || !aligned16(dy) || !aligned16(dx)) return BNS_ERR_ALIGN;
    if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) || workspace_bytes < np.total)
        return BNS_ERR_WORKSPACE;
    return backward_nhwc_impl(np, sampling, x, dy, gamma, mean, invstd, dx, dgamma, dbeta, workspace,
                              static_cast<cudaStream_t>(cuda_stream));
}

// ---------------------------------------------------------------------------------------- no-allocation forward
// Scratch for bns_forward_static: a fixed array in device memory that is part of the loaded library
// image, so a caller that has no way to obtain device memory of its own can still run the forward.
// The name below is only a host-side handle; the address the kernels need is looked up per device.
#define BNS_STATIC_WORKSPACE_BYTES (4u << 20)
static __device__ __align__(256) unsigned char g_static_workspace[BNS_STATIC_WORKSPACE_BYTES];

namespace {
void* g_static_workspace_address[kMaxDevices] = {};  // resolved by the first call made on each device
std::mutex g_static_workspace_mutex;                 // host threads may make that first call together

// Device address of the static scratch on the device that is current now.  The address is kept for the
// life of the process: it belongs to the device's primary context, which is assumed to live that long.
bns_status static_workspace_address(void** address) {
    int device = -1;
    if (cudaGetDevice(&device) != cudaSuccess) return BNS_ERR_CUDA;
    if (device < 0 || device >= kMaxDevices) return BNS_ERR_CUDA;
    std::lock_guard<std::mutex> guard(g_static_workspace_mutex);
    if (!g_static_workspace_address[device]) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_workspace) != cudaSuccess || !p) return BNS_ERR_CUDA;
        g_static_workspace_address[device] = p;
    }
    *address = g_static_workspace_address[device];
    return BNS_OK;
}
}  // namespace

size_t bns_static_workspace_bytes(void) { return BNS_STATIC_WORKSPACE_BYTES; }

bns_status bns_forward_static(const bns_shape* shape, const void* x, const float* gamma, const float* beta, float eps,
                              const bns_sampling* sampling, void* y, float* mean, float* invstd, void* cuda_stream) {
    Problem pb;
    bns_status st = make_problem(shape, sampling, pb);
    if (st != BNS_OK) return st;
    if (!x || !gamma || !beta || !y || !mean || !invstd) return BNS_ERR_NULL;
    if (!(eps > 0.f)) return BNS_ERR_SHAPE;
    if (!aligned16(x) || !aligned16(y)) return BNS_ERR_ALIGN;
    if (pb.total > BNS_STATIC_WORKSPACE_BYTES) return BNS_ERR_WORKSPACE;  // needs more scratch than is built in
    void* workspace = nullptr;
    st = static_workspace_address(&workspace);
    if (st != BNS_OK) return st;
    // Nothing in the scratch has to start at zero except the status word, which forward_impl clears itself
    // whenever a kernel may set it; every partial sum is written before it is read.
    return forward_impl(pb, sampling, x, gamma, beta, eps, y, mean, invstd, workspace,
                        static_cast<cudaStream_t>(cuda_stream));
}

}  // extern "C"

// One launch per direction for layers whose per-channel data fits on chip (sm_100a).
//
// A thread-block cluster of R blocks owns a group of G neighbouring channels.  In every sample row the
// group's data is one contiguous segment of Wd = G*H*W elements, a multiple of 16 bytes, so a row
// segment travels as one bulk asynchronous copy (cp.async.bulk + mbarrier).  Block r of the cluster
// loads the segments of its share of the N samples into shared memory: the "slab".  Everything else
// happens on the resident copy:
//   forward   statistics of the sampled set (one pass over shared memory of sums shifted by a pivot that is
//             itself a sampled value of the channel), combined across the cluster's blocks through
//             distributed shared memory in rank order (Chan's merge; every block computes the same
//             bits), then y = a x + b in place and bulk stores of the rows;
//   backward  sum dy and sum dy (x - mean) over every element, combined the same way, then the final
//             gradient of every element, sampled or not, written once (Eq. 6, both branches).
// x (and dy) are read from HBM once and y (dx) written once: 2 and 3 tensor passes, one launch each,
// no partial sums in global memory, no second launch to combine them.  Full BN runs through the same
// kernels with S = everything.
//
// Threads keep the position-space scheme of the streaming kernels: a thread owns V consecutive
// positions (16 bytes) of the segment and one of RL "row lanes"; it walks the rows rl, rl+RL, ... of
// the slab with per-position accumulators.  Waits on the copy barrier are bounded: a wait that runs
// out bumps a counter (bns_wait_timeouts) and the block carries on, so a kernel always ends.
#pragma once

#include <cooperative_groups.h>

#include "bns_kernels.cuh"

namespace bns {

namespace cg = cooperative_groups;

constexpr int kWarps = kThreads / 32;
constexpr int kSlabMaxChannels = 64;       // most channels per cluster
constexpr unsigned kWaitPolls = 1u << 22;  // mbarrier.try_wait attempts before a wait gives up

// Waits that ran out since the library was loaded (never reset by the kernels).
__device__ unsigned g_wait_timeouts;

// ------------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ unsigned shared_address(const void* p) {
    return static_cast<unsigned>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void barrier_init(uint64_t* bar, unsigned arrivals) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(shared_address(bar)), "r"(arrivals) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void barrier_expect_bytes(uint64_t* bar, unsigned bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(shared_address(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool barrier_try_wait(uint64_t* bar, unsigned parity) {
    unsigned done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(shared_address(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait for phase `parity` of the barrier; false (and the counter bumped) if it ran out.
__device__ __forceinline__ bool barrier_wait(uint64_t* bar, unsigned parity) {
    for (unsigned i = 0; i < kWaitPolls; ++i)
        if (barrier_try_wait(bar, parity)) return true;
    if ((threadIdx.x & 31) == 0) atomicAdd(&g_wait_timeouts, 1u);
    return false;
}
// global -> shared, `bytes` a multiple of 16, both addresses 16-byte aligned; completion is counted on `bar`
__device__ __forceinline__ void bulk_load(void* dst_shared, const void* src_global, unsigned bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     shared_address(dst_shared)),
                 "l"(src_global), "r"(bytes), "r"(shared_address(bar))
                 : "memory");
}
// shared -> global
__device__ __forceinline__ void bulk_store(void* dst_global, const void* src_shared, unsigned bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst_global),
                 "r"(shared_address(src_shared)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_store_commit_and_wait() {
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
}
// makes this thread's shared-memory writes visible to the bulk-copy engine
__device__ __forceinline__ void fence_shared_for_bulk() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire;" ::: "memory"); }

// ------------------------------------------------------------------------------------ geometry
// Filled by the host planner; all sizes in elements unless named bytes.
struct SlabGeom {
    int N, C, H, W, HW;
    int G;         // channels per group (C % G == 0)
    int Wd;        // G*HW: positions of a row segment
    int NV;        // Wd / V vectors per segment (<= kThreads)
    int RL;        // row lanes: kThreads / NV
    int R;         // blocks per cluster; block r holds samples [r*N/R, (r+1)*N/R)
    int rows_max;  // most samples any block holds
    unsigned P;    // C*HW
    unsigned row_bytes;
    // shared memory layout: byte offsets from the 128-byte aligned base
    unsigned off_x, off_g, off_fold, off_slices, off_part, off_all, off_coef, off_flag, off_origin, total_bytes;
};

// The sampling rule as the slab kernels see it.
struct SlabSel {
    int rule;              // bns_rule
    const int* list;       // BATCH: device list or NULL for begin .. begin+count-1
    int begin, count;
    PatchRule patch;       // FEATURE
    int nv, xv_is_bf16;    // VIRTUAL
    const void* xv;
    void* yv;
    const void* dyv;
    void* dxv;
    float inv_s;           // 1 / (sampled elements per channel)
};

enum { kSelNone = 0, kSelStatic = 1, kSelRows = 2, kSelOrigins = 3 };

// A thread's fixed view of the segment: which vector, which row lane, and for each of its V positions
// the channel (within the group) and the pixel.
template <int V>
struct SlabThread {
    bool active;
    int vc, rl;
    int g[V];
    int hw[V];             // (h << 16) | w
    unsigned static_bits;  // selection bits that do not depend on the row (kSelStatic)
    __device__ __forceinline__ SlabThread(const SlabGeom& geo) {
        rl = threadIdx.x / geo.NV;
        vc = threadIdx.x - rl * geo.NV;
        active = rl < geo.RL;
        const int p = vc * V;
        int c = p / geo.HW;
        const int i = p - c * geo.HW;
        int h = i / geo.W;
        int w = i - h * geo.W;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            g[j] = c;
            hw[j] = (h << 16) | w;
            if (++w == geo.W) {
                w = 0;
                if (++h == geo.H) {
                    h = 0;
                    ++c;
                }
            }
        }
        static_bits = 0;
    }
};

// How a block decides, per row of its slab, which of a thread's positions are sampled.
struct SlabSelState {
    int mode;
    const unsigned char* row_flag;  // kSelRows: 1 for a sampled row
    const int2* origin;             // kSelOrigins: clamped patch origin per row (stride 1) or per (row, channel)
    int origin_stride;              // 1 or G
    int ph, pw;
    int first_row;                  // first row of the slab that holds sampled elements (-1: none)
    int first_pixel;                // kSelStatic: pixel of a sampled element of that row
};

template <int V>
__device__ __forceinline__ unsigned selection_bits(const SlabSelState& st, const SlabThread<V>& me, int row) {
    if (st.mode == kSelRows) return st.row_flag[row] ? (1u << V) - 1u : 0u;
    if (st.mode == kSelOrigins) {
        unsigned bits = 0;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const int2 o = st.origin[row * st.origin_stride + (st.origin_stride > 1 ? me.g[j] : 0)];
            const int h = me.hw[j] >> 16, w = me.hw[j] & 0xffff;
            bits |= static_cast<unsigned>(h >= o.x && h < o.x + st.ph && w >= o.y && w < o.y + st.pw) << j;
        }
        return bits;
    }
    return me.static_bits;
}

// Prepares the selection state of this block (rows [n0, n0+rows) of channels [c0, c0+G)) and returns
// the number of sampled elements per channel among them.  Ends with a block barrier.
template <int V>
__device__ __forceinline__ float slab_prepare_selection(const SlabGeom& geo, const SlabSel& sel, unsigned char* smem,
                                                        int n0, int rows, int c0, SlabThread<V>& me, SlabSelState& st,
                                                        unsigned* status) {
    st.mode = kSelNone;
    st.row_flag = smem + geo.off_flag;
    st.origin = reinterpret_cast<const int2*>(smem + geo.off_origin);
    st.origin_stride = 1;
    st.ph = sel.patch.ph;
    st.pw = sel.patch.pw;
    st.first_row = 0;
    st.first_pixel = 0;
    float local = 0.f;
    if (sel.rule == 0) {  // FULL
        st.mode = kSelStatic;
        me.static_bits = (1u << V) - 1u;
        local = static_cast<float>(rows) * geo.HW;
    } else if (sel.rule == 1) {  // BATCH
        st.mode = kSelRows;
        unsigned char* flag = smem + geo.off_flag;
        int mine = 0;
        if (sel.list) {
            int* s_first = reinterpret_cast<int*>(smem + geo.off_origin);  // no patch origins under this rule
            for (int r = threadIdx.x; r < rows; r += kThreads) flag[r] = 0;
            if (threadIdx.x == 0) *s_first = 0x7fffffff;
            __syncthreads();
            // the list holds distinct samples, so the count of list entries in range is the count of sampled rows
            for (int j0 = 0; j0 < sel.count; j0 += kThreads) {
                const int j = j0 + threadIdx.x;
                const int n = j < sel.count ? sel.list[j] - n0 : -1;
                const bool in = n >= 0 && n < rows;
                if (in) {
                    flag[n] = 1;
                    atomicMin(s_first, n);
                }
                mine += __syncthreads_count(in);
            }
            st.first_row = mine ? *s_first : -1;
        } else {
            for (int r = threadIdx.x; r < rows; r += kThreads)
                flag[r] = (n0 + r >= sel.begin && n0 + r < sel.begin + sel.count) ? 1 : 0;
            const int lo = max(n0, sel.begin), hi = min(n0 + rows, sel.begin + sel.count);
            mine = max(0, hi - lo);
            st.first_row = mine ? lo - n0 : -1;
        }
        local = static_cast<float>(mine) * geo.HW;
    } else if (sel.rule == 2) {  // FEATURE
        local = static_cast<float>(rows) * sel.patch.ph * sel.patch.pw;
        if (!sel.patch.offsets) {
            st.mode = kSelStatic;
            st.first_pixel = sel.patch.oh * geo.W + sel.patch.ow;
            unsigned bits = 0;
#pragma unroll
            for (int j = 0; j < V; ++j) {
                const int h = me.hw[j] >> 16, w = me.hw[j] & 0xffff;
                bits |= static_cast<unsigned>(h >= sel.patch.oh && h < sel.patch.oh + sel.patch.ph &&
                                              w >= sel.patch.ow && w < sel.patch.ow + sel.patch.pw)
                        << j;
            }
            me.static_bits = bits;
        } else {
            st.mode = kSelOrigins;
            st.origin_stride = sel.patch.stride_c ? geo.G : 1;
            int2* origin = reinterpret_cast<int2*>(smem + geo.off_origin);
            const int entries = rows * st.origin_stride;
            for (int e = threadIdx.x; e < entries; e += kThreads) {
                const int r = e / st.origin_stride, g = e - r * st.origin_stride;
                int oh, ow;
                patch_origin(sel.patch, n0 + r, c0 + g, geo.H, geo.W, status, oh, ow);
                origin[e] = make_int2(oh, ow);
            }
        }
    } else {
        st.first_row = -1;
    }
    __syncthreads();
    return local;
}

// Pixel (inside the map of channel g) of a sampled element of row st.first_row: the pivot of the shifted sums.
__device__ __forceinline__ int slab_pivot_pixel(const SlabSelState& st, const SlabGeom& geo, int g) {
    if (st.mode == kSelOrigins) {
        const int2 o = st.origin[st.first_row * st.origin_stride + (st.origin_stride > 1 ? g : 0)];
        return o.x * geo.W + o.y;
    }
    return st.first_pixel;
}

// Per-channel totals of values kept per position.  The owner of positions [vc*V, vc*V+V) in row lane rl
// has stored acc[k][j] at s_fold[k*span + rl*Wd + vc*V + j] and the block has synchronised.  Warp
// (g, slice) adds its share of channel g's lanes*HW entries in a fixed order and leaves
// s_slices[(g*wpc + slice)*K + k]; after the next block barrier slab_total() adds the slices in index
// order, so every reader gets the same bits.
__device__ __forceinline__ int slab_warps_per_channel(const SlabGeom& geo) { return geo.G >= kWarps ? 1 : kWarps / geo.G; }

template <int K>
__device__ __forceinline__ void slab_reduce(const SlabGeom& geo, int lanes, int span, const float* s_fold, float* s_slices) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wpc = slab_warps_per_channel(geo);
    for (int g = warp / wpc; g < geo.G; g += kWarps / wpc) {
        const int slice = warp - (warp / wpc) * wpc;
        float tot[K];
#pragma unroll
        for (int k = 0; k < K; ++k) tot[k] = 0.f;
        for (int rl = 0; rl < lanes; ++rl) {
            const float* base = s_fold + rl * geo.Wd + g * geo.HW;
#pragma unroll 4
            for (int i = slice * 32 + lane; i < geo.HW; i += wpc * 32) {
#pragma unroll
                for (int k = 0; k < K; ++k) tot[k] += base[k * span + i];
            }
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
#pragma unroll
            for (int k = 0; k < K; ++k) tot[k] += __shfl_xor_sync(0xffffffffu, tot[k], d);
        }
        if (lane == 0) {
#pragma unroll
            for (int k = 0; k < K; ++k) s_slices[(g * wpc + slice) * K + k] = tot[k];
        }
    }
}

template <int K>
__device__ __forceinline__ float slab_total(const SlabGeom& geo, const float* s_slices, int g, int k) {
    const int wpc = slab_warps_per_channel(geo);
    float t = 0.f;
    for (int s = 0; s < wpc; ++s) t += s_slices[(g * wpc + s) * K + k];
    return t;
}

template <int V, int K>
__device__ __forceinline__ void slab_scatter(const SlabGeom& geo, const SlabThread<V>& me, const float (&acc)[K][V],
                                             float* s_fold) {
    if (!me.active) return;
    const int span = geo.RL * geo.Wd;
#pragma unroll
    for (int k = 0; k < K; ++k) {
        float4* dst = reinterpret_cast<float4*>(s_fold + k * span + me.rl * geo.Wd + me.vc * V);
#pragma unroll
        for (int q = 0; q < V / 4; ++q)
            dst[q] = make_float4(acc[k][4 * q], acc[k][4 * q + 1], acc[k][4 * q + 2], acc[k][4 * q + 3]);
    }
}

// A bulk copy takes a warp tens of cycles to issue, so the rows are dealt out across the warps: row r is
// issued by lane r / kWarps of warp r % kWarps (then by the same thread again every kThreads rows).
__device__ __forceinline__ int slab_first_issue_row() { return static_cast<int>(threadIdx.x >> 5) + static_cast<int>(threadIdx.x & 31) * kWarps; }

// Issues the bulk loads of this block's rows of one tensor; the barrier was told to expect all bytes.
template <typename S>
__device__ __forceinline__ void slab_issue_loads(const SlabGeom& geo, uint64_t* bar, S* dst, const S* src, int rows) {
    for (int r = slab_first_issue_row(); r < rows; r += kThreads)
        bulk_load(dst + static_cast<size_t>(r) * geo.Wd, src + static_cast<size_t>(r) * geo.P, geo.row_bytes, bar);
}

// Scalar element of the virtual samples (their type may differ from the real tensor's).
__device__ __forceinline__ float virtual_element(const void* base, int is_bf16, size_t at) {
    return is_bf16 ? to_float<BF16>(static_cast<const unsigned short*>(base)[at])
                   : static_cast<const float*>(base)[at];
}
__device__ __forceinline__ void store_virtual_element(void* base, int is_bf16, size_t at, float v) {
    if (is_bf16)
        static_cast<unsigned short*>(base)[at] = from_float<BF16>(v);
    else
        static_cast<float*>(base)[at] = v;
}

// Reads the partials that the R blocks of the cluster left at `mine` (G entries of type P each) into
// s_all[r*G + g], one remote read per thread, all in flight together.  Call after cluster.sync();
// ends with a block barrier and this block's arrival at the cluster barrier (it reads its peers no more).
template <typename P>
__device__ __forceinline__ void slab_gather_partials(cg::cluster_group& cluster, const SlabGeom& geo, P* mine, P* s_all) {
    for (int e = threadIdx.x; e < geo.R * geo.G; e += kThreads) {
        const int r = e / geo.G, g = e - r * geo.G;
        s_all[e] = *cluster.map_shared_rank(&mine[g], r);
    }
    __syncthreads();
    cluster_arrive();
}

// ------------------------------------------------------------------------------------ forward
template <typename T>
__global__ void __launch_bounds__(kThreads)
slab_forward_kernel(const typename T::storage* __restrict__ x, typename T::storage* __restrict__ y,
                    const float* __restrict__ gamma, const float* __restrict__ beta, float eps, SlabGeom geo, SlabSel sel,
                    float* __restrict__ mean, float* __restrict__ invstd, unsigned* status, MovingAverage ma) {
    using S = typename T::storage;
    constexpr int V = 16 / sizeof(S);
    extern __shared__ __align__(128) unsigned char smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = static_cast<int>(cluster.block_rank());
    const int group = blockIdx.x / geo.R;
    const int c0 = group * geo.G;
    const int n0 = static_cast<int>(static_cast<long long>(rank) * geo.N / geo.R);
    const int rows = static_cast<int>(static_cast<long long>(rank + 1) * geo.N / geo.R) - n0;
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem);
    S* sx = reinterpret_cast<S*>(smem + geo.off_x);
    float* s_fold = reinterpret_cast<float*>(smem + geo.off_fold);
    float* s_slices = reinterpret_cast<float*>(smem + geo.off_slices);
    float4* s_part = reinterpret_cast<float4*>(smem + geo.off_part);
    float4* s_all = reinterpret_cast<float4*>(smem + geo.off_all);
    float2* s_coef = reinterpret_cast<float2*>(smem + geo.off_coef);

    if (threadIdx.x == 0) barrier_init(bar, 1);
    __syncthreads();
    grid_dependency_wait();
    grid_dependency_launch();
    // (a copy may complete before the expectation is posted: the barrier's byte count then dips below zero
    // for a moment, but its phase cannot end before thread 0's arrival, which comes with the expectation)
    if (threadIdx.x == 0) barrier_expect_bytes(bar, static_cast<unsigned>(rows) * geo.row_bytes);
    slab_issue_loads<S>(geo, bar, sx, x + static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW, rows);
    // parameters of the channel this thread will finish, requested before anything waits
    float my_gamma = 0.f, my_beta = 0.f;
    if (threadIdx.x < geo.G) {
        my_gamma = gamma[c0 + threadIdx.x];
        my_beta = beta[c0 + threadIdx.x];
    }
    SlabThread<V> me(geo);
    SlabSelState st;
    const float local_count = slab_prepare_selection<V>(geo, sel, smem, n0, rows, c0, me, st, status);
    int lanes = geo.RL;            // row lanes whose sums take part in the fold
    const int span = geo.RL * geo.Wd;
    bool have_pivot = false;
    bool loaded = false;

    // Shifted sums of the sampled elements: s1 = sum (x - K), s2 = sum (x - K)^2 with the pivot K of a
    // channel one of its own sampled values, so nothing large is squared or cancelled.
    if (sel.rule == 3) {
        lanes = 1;
        if (rank == 0) {
            // VIRTUAL: the statistics come from xv alone; block 0 of the cluster takes them
            for (int p = threadIdx.x; p < geo.Wd; p += kThreads) {
                const int g = p / geo.HW;
                const size_t at = static_cast<size_t>(c0) * geo.HW + p;
                const float K = virtual_element(sel.xv, sel.xv_is_bf16, static_cast<size_t>(c0 + g) * geo.HW);
                float s1 = 0.f, s2 = 0.f;
                for (int v = 0; v < sel.nv; ++v) {
                    const float d = virtual_element(sel.xv, sel.xv_is_bf16, v * static_cast<size_t>(geo.P) + at) - K;
                    s1 += d;
                    s2 = fmaf(d, d, s2);
                }
                s_fold[p] = s1;
                s_fold[span + p] = s2;
            }
            have_pivot = true;
        }
    } else {
        barrier_wait(bar, 0);
        loaded = true;
        have_pivot = st.first_row >= 0;
        float acc[2][V];
#pragma unroll
        for (int j = 0; j < V; ++j) acc[0][j] = acc[1][j] = 0.f;
        if (me.active && have_pivot && !(st.mode == kSelStatic && me.static_bits == 0)) {
            float K[V];
#pragma unroll
            for (int j = 0; j < V; ++j)
                K[j] = to_float<T>(sx[static_cast<size_t>(st.first_row) * geo.Wd + me.g[j] * geo.HW + slab_pivot_pixel(st, geo, me.g[j])]);
            const S* mine = sx + me.vc * V;
            if (st.mode == kSelStatic) {
                const unsigned bits = me.static_bits;
                int row = me.rl;
                for (; row + 3 * geo.RL < rows; row += 4 * geo.RL) {
                    Vec<T, V> v[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) v[u].load(mine + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        float f[V];
                        v[u].unpack(f);
#pragma unroll
                        for (int j = 0; j < V; ++j) {
                            const float d = (bits >> j & 1u) ? f[j] - K[j] : 0.f;
                            acc[0][j] += d;
                            acc[1][j] = fmaf(d, d, acc[1][j]);
                        }
                    }
                }
                for (; row < rows; row += geo.RL) {
                    Vec<T, V> v;
                    v.load(mine + static_cast<size_t>(row) * geo.Wd);
                    float f[V];
                    v.unpack(f);
#pragma unroll
                    for (int j = 0; j < V; ++j) {
                        const float d = (bits >> j & 1u) ? f[j] - K[j] : 0.f;
                        acc[0][j] += d;
                        acc[1][j] = fmaf(d, d, acc[1][j]);
                    }
                }
            } else {
                for (int row = me.rl; row < rows; row += geo.RL) {
                    const unsigned bits = selection_bits<V>(st, me, row);
                    if (!bits) continue;
                    Vec<T, V> v;
                    v.load(mine + static_cast<size_t>(row) * geo.Wd);
                    float f[V];
                    v.unpack(f);
#pragma unroll
                    for (int j = 0; j < V; ++j) {
                        const float d = (bits >> j & 1u) ? f[j] - K[j] : 0.f;
                        acc[0][j] += d;
                        acc[1][j] = fmaf(d, d, acc[1][j]);
                    }
                }
            }
        }
        slab_scatter<V, 2>(geo, me, acc, s_fold);
    }
    __syncthreads();
    slab_reduce<2>(geo, lanes, span, s_fold, s_slices);
    __syncthreads();
    if (threadIdx.x < geo.G) {
        Moments m = {0.f, 0.f, 0.f};
        if (have_pivot) {
            float K;
            if (sel.rule == 3) {
                K = virtual_element(sel.xv, sel.xv_is_bf16, static_cast<size_t>(c0 + threadIdx.x) * geo.HW);
                m.cnt = static_cast<float>(sel.nv) * geo.HW;
            } else {
                K = to_float<T>(sx[static_cast<size_t>(st.first_row) * geo.Wd + threadIdx.x * geo.HW +
                                   slab_pivot_pixel(st, geo, threadIdx.x)]);
                m.cnt = local_count;
            }
            const float s1 = slab_total<2>(geo, s_slices, threadIdx.x, 0), s2 = slab_total<2>(geo, s_slices, threadIdx.x, 1);
            const float d = s1 / m.cnt;
            m.mean = K + d;
            m.m2 = fmaxf(s2 - s1 * d, 0.f);
        }
        s_part[threadIdx.x] = make_float4(m.cnt, m.mean, m.m2, 0.f);
    }
    // combine across the cluster: every block merges all blocks' moments in rank order
    cluster.sync();
    slab_gather_partials(cluster, geo, s_part, s_all);
    if (threadIdx.x < geo.G) {
        Moments all = {0.f, 0.f, 0.f};
        for (int r = 0; r < geo.R; ++r) {
            const float4 v = s_all[r * geo.G + threadIdx.x];
            all = merge(all, Moments{v.x, v.y, v.z});
        }
        const float is = 1.0f / sqrtf(all.m2 * sel.inv_s + eps);
        const float a = my_gamma * is;
        s_coef[threadIdx.x] = make_float2(a, fmaf(-all.mean, a, my_beta));
        if (rank == 0) {
            mean[c0 + threadIdx.x] = all.mean;
            invstd[c0 + threadIdx.x] = is;
            ma.update(c0 + threadIdx.x, all.mean, all.m2 * sel.inv_s);
        }
    }
    __syncthreads();
    if (!loaded) barrier_wait(bar, 0);
    // normalise + affine on the resident rows, in place
    if (me.active) {
        float a[V], b[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float2 k = s_coef[me.g[j]];
            a[j] = k.x;
            b[j] = k.y;
        }
        S* mine = sx + me.vc * V;
        int row = me.rl;
        for (; row + 3 * geo.RL < rows; row += 4 * geo.RL) {
            Vec<T, V> v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u].load(mine + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                float f[V];
                v[u].unpack(f);
#pragma unroll
                for (int j = 0; j < V; ++j) f[j] = fmaf(a[j], f[j], b[j]);
                v[u].pack(f);
                v[u].store(mine + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
            }
        }
        for (; row < rows; row += geo.RL) {
            S* at = mine + static_cast<size_t>(row) * geo.Wd;
            Vec<T, V> v;
            v.load(at);
            float f[V];
            v.unpack(f);
#pragma unroll
            for (int j = 0; j < V; ++j) f[j] = fmaf(a[j], f[j], b[j]);
            v.pack(f);
            v.store(at);
        }
    }
    fence_shared_for_bulk();
    __syncthreads();
    {
        S* dst = y + static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW;
        for (int r = slab_first_issue_row(); r < rows; r += kThreads)
            bulk_store(dst + static_cast<size_t>(r) * geo.P, sx + static_cast<size_t>(r) * geo.Wd, geo.row_bytes);
    }
    if (sel.rule == 3 && sel.yv && rank == 0) {
        // the same map applied to the virtual samples of this channel group
        const int total = sel.nv * geo.Wd;
        for (int e = threadIdx.x; e < total; e += kThreads) {
            const int v = e / geo.Wd, p = e - v * geo.Wd;
            const float2 k = s_coef[p / geo.HW];
            const size_t at = v * static_cast<size_t>(geo.P) + static_cast<size_t>(c0) * geo.HW + p;
            store_virtual_element(sel.yv, sel.xv_is_bf16, at, fmaf(k.x, virtual_element(sel.xv, sel.xv_is_bf16, at), k.y));
        }
    }
    bulk_store_commit_and_wait();
    cluster_wait();  // no block leaves while a peer may still read its shared memory
}

// ------------------------------------------------------------------------------------ backward
template <typename T>
__global__ void __launch_bounds__(kThreads)
slab_backward_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                     typename T::storage* __restrict__ dx, const float* __restrict__ gamma,
                     const float* __restrict__ mean, const float* __restrict__ invstd, SlabGeom geo, SlabSel sel,
                     float* __restrict__ dgamma, float* __restrict__ dbeta, unsigned* status) {
    using S = typename T::storage;
    constexpr int V = 16 / sizeof(S);
    extern __shared__ __align__(128) unsigned char smem[];
    cg::cluster_group cluster = cg::this_cluster();
    const int rank = static_cast<int>(cluster.block_rank());
    const int group = blockIdx.x / geo.R;
    const int c0 = group * geo.G;
    const int n0 = static_cast<int>(static_cast<long long>(rank) * geo.N / geo.R);
    const int rows = static_cast<int>(static_cast<long long>(rank + 1) * geo.N / geo.R) - n0;
    uint64_t* bar = reinterpret_cast<uint64_t*>(smem);
    S* sx = reinterpret_cast<S*>(smem + geo.off_x);
    S* sg = reinterpret_cast<S*>(smem + geo.off_g);
    float* s_fold = reinterpret_cast<float*>(smem + geo.off_fold);
    float* s_slices = reinterpret_cast<float*>(smem + geo.off_slices);
    float2* s_part = reinterpret_cast<float2*>(smem + geo.off_part);
    float2* s_all = reinterpret_cast<float2*>(smem + geo.off_all);
    float4* s_coef = reinterpret_cast<float4*>(smem + geo.off_coef);  // (a, A, Q, mean) per channel

    if (threadIdx.x == 0) barrier_init(bar, 1);
    __syncthreads();
    grid_dependency_wait();
    grid_dependency_launch();
    if (threadIdx.x == 0) barrier_expect_bytes(bar, 2u * static_cast<unsigned>(rows) * geo.row_bytes);
    {
        const size_t first = static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW;
        slab_issue_loads<S>(geo, bar, sx, x + first, rows);
        slab_issue_loads<S>(geo, bar, sg, dy + first, rows);
    }
    float my_gamma = 0.f, my_mean = 0.f, my_invstd = 0.f;
    if (threadIdx.x < geo.G) {
        my_gamma = gamma[c0 + threadIdx.x];
        my_mean = mean[c0 + threadIdx.x];
        my_invstd = invstd[c0 + threadIdx.x];
    }
    SlabThread<V> me(geo);
    SlabSelState st;
    slab_prepare_selection<V>(geo, sel, smem, n0, rows, c0, me, st, status);
    const int span = geo.RL * geo.Wd;
    float mu[V];
#pragma unroll
    for (int j = 0; j < V; ++j) mu[j] = mean[c0 + me.g[j]];
    barrier_wait(bar, 0);

    // sums of Eq. 5 over every resident element
    {
        float acc[2][V];
#pragma unroll
        for (int j = 0; j < V; ++j) acc[0][j] = acc[1][j] = 0.f;
        if (me.active) {
            const S* mx = sx + me.vc * V;
            const S* mg = sg + me.vc * V;
            int row = me.rl;
            for (; row + 3 * geo.RL < rows; row += 4 * geo.RL) {
                Vec<T, V> vx[4], vg[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    vx[u].load(mx + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
                    vg[u].load(mg + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float fx[V], fg[V];
                    vx[u].unpack(fx);
                    vg[u].unpack(fg);
#pragma unroll
                    for (int j = 0; j < V; ++j) {
                        acc[0][j] += fg[j];
                        acc[1][j] = fmaf(fg[j], fx[j] - mu[j], acc[1][j]);
                    }
                }
            }
            for (; row < rows; row += geo.RL) {
                Vec<T, V> vx, vg;
                vx.load(mx + static_cast<size_t>(row) * geo.Wd);
                vg.load(mg + static_cast<size_t>(row) * geo.Wd);
                float fx[V], fg[V];
                vx.unpack(fx);
                vg.unpack(fg);
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    acc[0][j] += fg[j];
                    acc[1][j] = fmaf(fg[j], fx[j] - mu[j], acc[1][j]);
                }
            }
        }
        slab_scatter<V, 2>(geo, me, acc, s_fold);
    }
    __syncthreads();
    if (sel.rule == 3 && sel.dyv && rank == 0) {
        // the virtual rows were normalised with the same statistics: their gradient joins the sums
        for (int p = threadIdx.x; p < geo.Wd; p += kThreads) {
            const size_t at = static_cast<size_t>(c0) * geo.HW + p;
            const float m = mean[c0 + p / geo.HW];
            float a0 = 0.f, a1 = 0.f;
            for (int v = 0; v < sel.nv; ++v) {
                const float gv = virtual_element(sel.dyv, sel.xv_is_bf16, v * static_cast<size_t>(geo.P) + at);
                a0 += gv;
                a1 = fmaf(gv, virtual_element(sel.xv, sel.xv_is_bf16, v * static_cast<size_t>(geo.P) + at) - m, a1);
            }
            s_fold[p] += a0;         // row lane 0 of position p
            s_fold[span + p] += a1;
        }
        __syncthreads();
    }
    slab_reduce<2>(geo, geo.RL, span, s_fold, s_slices);
    __syncthreads();
    if (threadIdx.x < geo.G)
        s_part[threadIdx.x] = make_float2(slab_total<2>(geo, s_slices, threadIdx.x, 0), slab_total<2>(geo, s_slices, threadIdx.x, 1));
    cluster.sync();
    slab_gather_partials(cluster, geo, s_part, s_all);
    if (threadIdx.x < geo.G) {
        float sum_dy = 0.f, sum_dyxc = 0.f;
        for (int r = 0; r < geo.R; ++r) {
            const float2 v = s_all[r * geo.G + threadIdx.x];
            sum_dy += v.x;
            sum_dyxc += v.y;
        }
        const float dg = sum_dyxc * my_invstd;
        const FixCoef k = fix_coef(my_gamma, my_mean, my_invstd, dg, sum_dy, sel.inv_s);
        s_coef[threadIdx.x] = make_float4(k.a, k.A, k.Q, k.mu);
        if (rank == 0) {
            dbeta[c0 + threadIdx.x] = sum_dy;
            dgamma[c0 + threadIdx.x] = dg;
        }
    }
    __syncthreads();
    // the gradient of every resident element: both branches of Eq. 6, written over dy's copy
    if (me.active) {
        float a[V], A[V], Q[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float4 k = s_coef[me.g[j]];
            a[j] = k.x;
            A[j] = k.y;
            Q[j] = k.z;
        }
        const S* mx = sx + me.vc * V;
        S* mg = sg + me.vc * V;
        if (st.mode == kSelStatic && me.static_bits == 0) {
            // no sampled element among this thread's positions: lower branch only, x is not needed
            int row = me.rl;
            for (; row + 3 * geo.RL < rows; row += 4 * geo.RL) {
                Vec<T, V> vg[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) vg[u].load(mg + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    float fg[V];
                    vg[u].unpack(fg);
#pragma unroll
                    for (int j = 0; j < V; ++j) fg[j] *= a[j];
                    vg[u].pack(fg);
                    vg[u].store(mg + static_cast<size_t>(row + u * geo.RL) * geo.Wd);
                }
            }
            for (; row < rows; row += geo.RL) {
                Vec<T, V> vg;
                vg.load(mg + static_cast<size_t>(row) * geo.Wd);
                float fg[V];
                vg.unpack(fg);
#pragma unroll
                for (int j = 0; j < V; ++j) fg[j] *= a[j];
                vg.pack(fg);
                vg.store(mg + static_cast<size_t>(row) * geo.Wd);
            }
        } else {
#pragma unroll 2
            for (int row = me.rl; row < rows; row += geo.RL) {
                const size_t at = static_cast<size_t>(row) * geo.Wd;
                const unsigned bits = selection_bits<V>(st, me, row);
                Vec<T, V> vg, vx;
                vg.load(mg + at);
                vx.load(mx + at);
                float fg[V], fx[V];
                vg.unpack(fg);
                vx.unpack(fx);
#pragma unroll
                for (int j = 0; j < V; ++j)
                    fg[j] = (bits >> j & 1u) ? fmaf(a[j], fg[j], -A[j]) - Q[j] * (fx[j] - mu[j]) : a[j] * fg[j];
                vg.pack(fg);
                vg.store(mg + at);
            }
        }
    }
    fence_shared_for_bulk();
    __syncthreads();
    {
        S* dst = dx + static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW;
        for (int r = slab_first_issue_row(); r < rows; r += kThreads)
            bulk_store(dst + static_cast<size_t>(r) * geo.P, sg + static_cast<size_t>(r) * geo.Wd, geo.row_bytes);
    }
    if (sel.rule == 3 && sel.dxv && rank == 0) {
        // upper branch of Eq. 6 for every virtual element of this channel group
        const int total = sel.nv * geo.Wd;
        for (int e = threadIdx.x; e < total; e += kThreads) {
            const int v = e / geo.Wd, p = e - v * geo.Wd;
            const float4 k = s_coef[p / geo.HW];
            const size_t at = v * static_cast<size_t>(geo.P) + static_cast<size_t>(c0) * geo.HW + p;
            const float gv = sel.dyv ? virtual_element(sel.dyv, sel.xv_is_bf16, at) : 0.f;
            const float xv = virtual_element(sel.xv, sel.xv_is_bf16, at);
            store_virtual_element(sel.dxv, sel.xv_is_bf16, at, fmaf(k.x, gv, -k.y) - k.z * (xv - k.w));
        }
    }
    bulk_store_commit_and_wait();
    cluster_wait();
}

}  // namespace bns

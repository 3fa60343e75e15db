// One launch per direction for layers whose per-channel data fits on chip (sm_100a).
//
// A thread-block cluster of R blocks owns a group of G neighbouring channels.  In every sample row the
// group's data is one contiguous segment of Wd = G*H*W elements, a multiple of 16 bytes, so a row
// segment travels as one bulk asynchronous copy (cp.async.bulk + mbarrier).  Block r of the cluster
// loads the segments of its share of the N samples into shared memory: the "slab".  Everything else
// happens on the resident copy:
//   forward   statistics of the sampled set (two passes over shared memory: local mean, then squared
//             deviations about it), combined across the cluster's blocks through distributed shared
//             memory in rank order (Chan's merge; every block computes the same bits), then
//             y = a x + b in place and bulk stores of the rows;
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
    unsigned off_x, off_g, off_fold, off_slices, off_part, off_coef, off_flag, off_origin, total_bytes;
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
        int p = vc * V;
        int c = p / geo.HW;
        int i = p - c * geo.HW;
#pragma unroll
        for (int j = 0; j < V; ++j) {
            g[j] = c;
            const int h = i / geo.W;
            hw[j] = (h << 16) | (i - h * geo.W);
            if (++i == geo.HW) {
                i = 0;
                ++c;
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
};

template <int V>
__device__ __forceinline__ unsigned selection_bits(const SlabSelState& st, const SlabThread<V>& me, int row) {
    if (st.mode == kSelStatic) return me.static_bits;
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
    return 0u;
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
            for (int r = threadIdx.x; r < rows; r += kThreads) flag[r] = 0;
            __syncthreads();
            for (int j = threadIdx.x; j < sel.count; j += kThreads) {
                const int n = sel.list[j] - n0;
                if (n >= 0 && n < rows) flag[n] = 1;
            }
            // the list holds distinct samples, so the count of set flags is the count of list entries in range
            for (int j0 = 0; j0 < sel.count; j0 += kThreads) {
                const int j = j0 + threadIdx.x;
                const int n = j < sel.count ? sel.list[j] - n0 : -1;
                mine += __syncthreads_count(n >= 0 && n < rows);
            }
        } else {
            for (int r = threadIdx.x; r < rows; r += kThreads)
                flag[r] = (n0 + r >= sel.begin && n0 + r < sel.begin + sel.count) ? 1 : 0;
            const int lo = max(n0, sel.begin), hi = min(n0 + rows, sel.begin + sel.count);
            mine = max(0, hi - lo);
        }
        local = static_cast<float>(mine) * geo.HW;
    } else if (sel.rule == 2) {  // FEATURE
        local = static_cast<float>(rows) * sel.patch.ph * sel.patch.pw;
        if (!sel.patch.offsets) {
            st.mode = kSelStatic;
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
    }
    __syncthreads();
    return local;
}

// Sums, per channel of the group, the per-position values acc[k][j] that the active threads hold:
// out[g*K + k].  Fixed order: row lanes and pixels are walked by (warp slice, lane) and combined by a
// shuffle tree, slices are added in index order.  Uses s_fold (K*RL*Wd floats) and s_slices; ends with
// a block barrier, after which `out` may be read by every thread.
template <int V, int K>
__device__ __forceinline__ void slab_fold(const SlabGeom& geo, const SlabThread<V>& me, const float (&acc)[K][V],
                                          float* s_fold, float* s_slices, float* out) {
    const int span = geo.RL * geo.Wd;
    if (me.active) {
#pragma unroll
        for (int k = 0; k < K; ++k) {
            float4* dst = reinterpret_cast<float4*>(s_fold + k * span + me.rl * geo.Wd + me.vc * V);
#pragma unroll
            for (int q = 0; q < V / 4; ++q) dst[q] = make_float4(acc[k][4 * q], acc[k][4 * q + 1], acc[k][4 * q + 2], acc[k][4 * q + 3]);
        }
    }
    __syncthreads();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int wpc = geo.G >= kWarps ? 1 : kWarps / geo.G;  // warps that share one channel
    for (int g = warp / wpc; g < geo.G; g += kWarps / wpc) {
        const int slice = warp - (warp / wpc) * wpc;
        float tot[K];
#pragma unroll
        for (int k = 0; k < K; ++k) tot[k] = 0.f;
        for (int rl = 0; rl < geo.RL; ++rl) {
            const float* base = s_fold + rl * geo.Wd + g * geo.HW;
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
    __syncthreads();
    for (int e = threadIdx.x; e < geo.G * K; e += kThreads) {
        const int g = e / K, k = e - g * K;
        float t = 0.f;
        for (int s = 0; s < wpc; ++s) t += s_slices[(g * wpc + s) * K + k];
        out[e] = t;
    }
    __syncthreads();
}

// Issues the bulk loads of this block's rows of one tensor (warp 0; the barrier expects all bytes).
template <typename S>
__device__ __forceinline__ void slab_issue_loads(const SlabGeom& geo, uint64_t* bar, S* dst, const S* src, int rows) {
    for (int r = threadIdx.x; r < rows; r += 32)
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

// ------------------------------------------------------------------------------------ forward
template <typename T>
__global__ void __launch_bounds__(kThreads)
slab_forward_kernel(const typename T::storage* __restrict__ x, typename T::storage* __restrict__ y,
                    const float* __restrict__ gamma, const float* __restrict__ beta, float eps, SlabGeom geo, SlabSel sel,
                    float* __restrict__ mean, float* __restrict__ invstd, unsigned* status) {
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
    float2* s_coef = reinterpret_cast<float2*>(smem + geo.off_coef);
    float* s_red = reinterpret_cast<float*>(smem + geo.off_coef) + 2 * geo.G;  // G floats of folded sums

    if (threadIdx.x == 0) barrier_init(bar, 1);
    __syncthreads();
    grid_dependency_wait();
    grid_dependency_launch();
    if (threadIdx.x < 32) {
        if (threadIdx.x == 0) barrier_expect_bytes(bar, static_cast<unsigned>(rows) * geo.row_bytes);
        __syncwarp();
        slab_issue_loads<S>(geo, bar, sx, x + static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW, rows);
    }
    SlabThread<V> me(geo);
    SlabSelState st;
    const float local_count = slab_prepare_selection<V>(geo, sel, smem, n0, rows, c0, me, st, status);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (sel.rule == 3) {
        // VIRTUAL: the statistics come from xv alone; block 0 of the cluster computes them (two passes
        // over the group's nv*HW elements per channel, one warp per channel), the others contribute nothing
        for (int g = warp; g < geo.G; g += kWarps) {
            Moments m = {0.f, 0.f, 0.f};
            if (rank == 0) {
                const size_t cb = static_cast<size_t>(c0 + g) * geo.HW;
                float sum = 0.f;
                for (int v = 0; v < sel.nv; ++v)
                    for (int i = lane; i < geo.HW; i += 32) sum += virtual_element(sel.xv, sel.xv_is_bf16, v * static_cast<size_t>(geo.P) + cb + i);
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
                m.cnt = static_cast<float>(sel.nv) * geo.HW;
                m.mean = sum / m.cnt;
                float dev = 0.f;
                for (int v = 0; v < sel.nv; ++v)
                    for (int i = lane; i < geo.HW; i += 32) {
                        const float d = virtual_element(sel.xv, sel.xv_is_bf16, v * static_cast<size_t>(geo.P) + cb + i) - m.mean;
                        dev = fmaf(d, d, dev);
                    }
#pragma unroll
                for (int d = 16; d > 0; d >>= 1) dev += __shfl_xor_sync(0xffffffffu, dev, d);
                m.m2 = dev;
            }
            if (lane == 0) s_part[g] = make_float4(m.cnt, m.mean, m.m2, 0.f);
        }
        barrier_wait(bar, 0);
    } else {
        barrier_wait(bar, 0);
        // local mean of the sampled elements, then their squared deviations about it
        float acc[1][V];
#pragma unroll
        for (int j = 0; j < V; ++j) acc[0][j] = 0.f;
        if (me.active) {
            for (int row = me.rl; row < rows; row += geo.RL) {
                const unsigned bits = selection_bits<V>(st, me, row);
                if (!bits) continue;
                Vec<T, V> v;
                v.load(sx + static_cast<size_t>(row) * geo.Wd + me.vc * V);
                float f[V];
                v.unpack(f);
#pragma unroll
                for (int j = 0; j < V; ++j) acc[0][j] += (bits >> j & 1u) ? f[j] : 0.f;
            }
        }
        slab_fold<V, 1>(geo, me, acc, s_fold, s_slices, s_red);
        float lmean[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            lmean[j] = local_count > 0.f ? s_red[me.g[j] < geo.G ? me.g[j] : 0] / local_count : 0.f;
            acc[0][j] = 0.f;
        }
        if (me.active) {
            for (int row = me.rl; row < rows; row += geo.RL) {
                const unsigned bits = selection_bits<V>(st, me, row);
                if (!bits) continue;
                Vec<T, V> v;
                v.load(sx + static_cast<size_t>(row) * geo.Wd + me.vc * V);
                float f[V];
                v.unpack(f);
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    const float d = f[j] - lmean[j];
                    acc[0][j] = fmaf((bits >> j & 1u) ? d : 0.f, d, acc[0][j]);
                }
            }
        }
        float* s_m2 = s_red + geo.G;
        if (threadIdx.x < geo.G) s_part[threadIdx.x].y = local_count > 0.f ? s_red[threadIdx.x] / local_count : 0.f;
        slab_fold<V, 1>(geo, me, acc, s_fold, s_slices, s_m2);
        if (threadIdx.x < geo.G) {
            s_part[threadIdx.x].x = local_count;
            s_part[threadIdx.x].z = s_m2[threadIdx.x];
            s_part[threadIdx.x].w = 0.f;
        }
    }
    // combine across the cluster: every block merges all blocks' moments in rank order
    cluster.sync();
    if (threadIdx.x < geo.G) {
        Moments all = {0.f, 0.f, 0.f};
        for (int r = 0; r < geo.R; ++r) {
            const float4 v = *cluster.map_shared_rank(&s_part[threadIdx.x], r);
            all = merge(all, Moments{v.x, v.y, v.z});
        }
        const int c = c0 + threadIdx.x;
        const float is = 1.0f / sqrtf(all.m2 * sel.inv_s + eps);
        const float a = gamma[c] * is;
        s_coef[threadIdx.x] = make_float2(a, fmaf(-all.mean, a, beta[c]));
        if (rank == 0) {
            mean[c] = all.mean;
            invstd[c] = is;
        }
    }
    cluster_arrive();  // this block is done reading its peers' shared memory
    __syncthreads();
    // normalise + affine on the resident rows, in place
    if (me.active) {
        float a[V], b[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float2 k = s_coef[me.g[j] < geo.G ? me.g[j] : 0];
            a[j] = k.x;
            b[j] = k.y;
        }
        for (int row = me.rl; row < rows; row += geo.RL) {
            S* at = sx + static_cast<size_t>(row) * geo.Wd + me.vc * V;
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
        for (int r = threadIdx.x; r < rows; r += kThreads)
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
    float4* s_coef = reinterpret_cast<float4*>(smem + geo.off_coef);  // (a, A, Q, mean) per channel

    if (threadIdx.x == 0) barrier_init(bar, 1);
    __syncthreads();
    grid_dependency_wait();
    grid_dependency_launch();
    if (threadIdx.x < 32) {
        if (threadIdx.x == 0) barrier_expect_bytes(bar, 2u * static_cast<unsigned>(rows) * geo.row_bytes);
        __syncwarp();
        const size_t first = static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW;
        slab_issue_loads<S>(geo, bar, sx, x + first, rows);
        slab_issue_loads<S>(geo, bar, sg, dy + first, rows);
    }
    SlabThread<V> me(geo);
    SlabSelState st;
    slab_prepare_selection<V>(geo, sel, smem, n0, rows, c0, me, st, status);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    float mu[V];
#pragma unroll
    for (int j = 0; j < V; ++j) mu[j] = mean[c0 + (me.g[j] < geo.G ? me.g[j] : 0)];
    barrier_wait(bar, 0);

    // sums of Eq. 5 over every resident element
    float acc[2][V];
#pragma unroll
    for (int j = 0; j < V; ++j) acc[0][j] = acc[1][j] = 0.f;
    if (me.active) {
        for (int row = me.rl; row < rows; row += geo.RL) {
            const size_t at = static_cast<size_t>(row) * geo.Wd + me.vc * V;
            Vec<T, V> vx, vg;
            vx.load(sx + at);
            vg.load(sg + at);
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
    slab_fold<V, 2>(geo, me, acc, s_fold, s_slices, reinterpret_cast<float*>(s_part));
    if (sel.rule == 3 && sel.dyv && rank == 0) {
        // the virtual rows were normalised with the same statistics: their gradient joins the sums
        for (int g = warp; g < geo.G; g += kWarps) {
            const size_t cb = static_cast<size_t>(c0 + g) * geo.HW;
            const float m = mean[c0 + g];
            float a0 = 0.f, a1 = 0.f;
            for (int v = 0; v < sel.nv; ++v)
                for (int i = lane; i < geo.HW; i += 32) {
                    const size_t at = v * static_cast<size_t>(geo.P) + cb + i;
                    const float gv = virtual_element(sel.dyv, sel.xv_is_bf16, at);
                    a0 += gv;
                    a1 = fmaf(gv, virtual_element(sel.xv, sel.xv_is_bf16, at) - m, a1);
                }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                a0 += __shfl_xor_sync(0xffffffffu, a0, d);
                a1 += __shfl_xor_sync(0xffffffffu, a1, d);
            }
            if (lane == 0) {
                s_part[g].x += a0;
                s_part[g].y += a1;
            }
        }
    }
    cluster.sync();
    if (threadIdx.x < geo.G) {
        float sum_dy = 0.f, sum_dyxc = 0.f;
        for (int r = 0; r < geo.R; ++r) {
            const float2 v = *cluster.map_shared_rank(&s_part[threadIdx.x], r);
            sum_dy += v.x;
            sum_dyxc += v.y;
        }
        const int c = c0 + threadIdx.x;
        const float is = invstd[c];
        const float dg = sum_dyxc * is;
        const FixCoef k = fix_coef(gamma[c], mean[c], is, dg, sum_dy, sel.inv_s);
        s_coef[threadIdx.x] = make_float4(k.a, k.A, k.Q, k.mu);
        if (rank == 0) {
            dbeta[c] = sum_dy;
            dgamma[c] = dg;
        }
    }
    cluster_arrive();
    __syncthreads();
    // the gradient of every resident element: both branches of Eq. 6, written over dy's copy
    if (me.active) {
        float a[V], A[V], Q[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float4 k = s_coef[me.g[j] < geo.G ? me.g[j] : 0];
            a[j] = k.x;
            A[j] = k.y;
            Q[j] = k.z;
        }
        for (int row = me.rl; row < rows; row += geo.RL) {
            const size_t at = static_cast<size_t>(row) * geo.Wd + me.vc * V;
            const unsigned bits = selection_bits<V>(st, me, row);
            Vec<T, V> vg;
            vg.load(sg + at);
            float fg[V];
            vg.unpack(fg);
            if (bits) {
                Vec<T, V> vx;
                vx.load(sx + at);
                float fx[V];
                vx.unpack(fx);
#pragma unroll
                for (int j = 0; j < V; ++j)
                    fg[j] = (bits >> j & 1u) ? fmaf(a[j], fg[j], -A[j]) - Q[j] * (fx[j] - mu[j]) : a[j] * fg[j];
            } else {
#pragma unroll
                for (int j = 0; j < V; ++j) fg[j] *= a[j];
            }
            vg.pack(fg);
            vg.store(sg + at);
        }
    }
    fence_shared_for_bulk();
    __syncthreads();
    {
        S* dst = dx + static_cast<size_t>(n0) * geo.P + static_cast<size_t>(c0) * geo.HW;
        for (int r = threadIdx.x; r < rows; r += kThreads)
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

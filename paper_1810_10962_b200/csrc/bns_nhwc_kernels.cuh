// Channels-last (NHWC) kernels of the BN-sampling library (sm_100a).
//
// The paper's own layout (Appendix A: B in R^{N x H x W x C}, statistics reduce dims 0,1,2).  A tensor is
// R = N*H*W rows of C contiguous channel values.  A thread owns V consecutive channels (up to 16 bytes)
// for the whole kernel and walks down rows; a block is CW channel-vectors wide and RL row-lanes deep, so
// one step of a block reads RL consecutive rows - contiguous memory when the block is as wide as a row.
// Per-channel sums stay in registers, are folded across the row-lanes through shared memory once per
// block, and the per-block partials (one per channel and block) are combined in a fixed order by the
// finalize kernels at the end of this file.  A sampled pixel is a whole contiguous channel vector here,
// which is what makes Feature Sampling cheap in this layout.
#pragma once

#include "bns_kernels.cuh"

namespace bns {

// Which rows of the tensor a kernel visits, enumerated q = 0 .. total-1.
struct RowSet {
    enum { kAll = 0, kSamples = 1, kPatches = 2 };
    int mode;
    int total;          // rows in the set
    const int* list;    // kSamples: sample indices (device) or NULL for begin .. begin+count-1
    int begin, HW;      // kSamples: row q belongs to sample q / HW
    PatchRule patch;    // kPatches: shared or per-sample location (never per map: a row spans all channels)
    int H, W;
    __device__ __forceinline__ int row(int q, unsigned* status) const {
        if (mode == kAll) return q;
        if (mode == kSamples) {
            const int i = q / HW;
            return (list ? list[i] : begin + i) * HW + (q - i * HW);
        }
        const int PP = patch.ph * patch.pw;
        const int n = q / PP, e = q - n * PP;
        const int r = e / patch.pw, col = e - r * patch.pw;
        int oh, ow;
        patch_origin(patch, n, 0, H, W, status, oh, ow);
        return n * (H * W) + (oh + r) * W + ow + col;
    }
};

// Block shape: CW channel-vectors wide, RL row-lanes deep; grid.y tiles the channel-vectors.
struct NhwcShape {
    int C, V_unused, CV, CW, RL;  // channels, -, vectors per row, vectors per block, row-lanes per block
    int rows_per_block;           // rows of the set that one block (grid.x) visits; a multiple of RL
};

struct NhwcThread {
    int cv, rl;    // channel-vector of the row, row-lane
    bool active;
    __device__ __forceinline__ NhwcThread(const NhwcShape& s) {
        const int t = threadIdx.x;
        const int cvi = t % s.CW;
        rl = t / s.CW;
        cv = blockIdx.y * s.CW + cvi;
        active = rl < s.RL && cv < s.CV;
    }
};

// ------------------------------------------------------------------------------------ statistics
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
nhwc_moments_kernel(const typename T::storage* __restrict__ x, RowSet set, NhwcShape s, float4* __restrict__ partials,
                    unsigned* status) {
    __shared__ float s_cnt[kThreads], s_mean[kThreads * V], s_m2[kThreads * V];
    grid_dependency_wait();
    grid_dependency_launch();
    const NhwcThread me(s);
    const int q0 = blockIdx.x * s.rows_per_block, q1 = min(set.total, q0 + s.rows_per_block);
    float K[V], s1[V], s2[V], cnt = 0.f;
#pragma unroll
    for (int j = 0; j < V; ++j) K[j] = s1[j] = s2[j] = 0.f;
    if (me.active) {
        const typename T::storage* xp = x + static_cast<size_t>(me.cv) * V;
        for (int q = q0 + me.rl; q < q1; q += kUnroll * s.RL) {
            Vec<T, V> v[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (q + u * s.RL < q1) v[u].load(xp + static_cast<size_t>(set.row(q + u * s.RL, status)) * s.C);
            if (cnt == 0.f) {
#pragma unroll
                for (int j = 0; j < V; ++j) K[j] = v[0].get(j);  // pivot: the thread's first row
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (q + u * s.RL < q1) {
#pragma unroll
                    for (int j = 0; j < V; ++j) {
                        float d = v[u].get(j) - K[j];
                        s1[j] += d;
                        s2[j] = fmaf(d, d, s2[j]);
                    }
                    cnt += 1.f;
                }
        }
    }
    s_cnt[threadIdx.x] = cnt;
#pragma unroll
    for (int j = 0; j < V; ++j) {
        Moments m = from_shifted_sums(cnt, K[j], s1[j], s2[j]);
        s_mean[threadIdx.x * V + j] = m.mean;
        s_m2[threadIdx.x * V + j] = m.m2;
    }
    __syncthreads();
    // channel ch of the block (ch < CW*V): merge its RL row-lane entries in lane order
    for (int ch = threadIdx.x; ch < s.CW * V; ch += kThreads) {
        const int cvi = ch / V, j = ch - cvi * V;
        const int c = (blockIdx.y * s.CW + cvi) * V + j;
        if (c >= s.C) continue;
        Moments acc = {0.f, 0.f, 0.f};
        for (int rl = 0; rl < s.RL; ++rl) {
            const int t = rl * s.CW + cvi;
            acc = merge(acc, Moments{s_cnt[t], s_mean[t * V + j], s_m2[t * V + j]});
        }
        partials[static_cast<size_t>(blockIdx.x) * s.C + c] = make_float4(acc.cnt, acc.mean, acc.m2, 0.f);
    }
}

// ------------------------------------------------------------------------------------ normalise + affine
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
nhwc_normalize_kernel(const typename T::storage* __restrict__ x, typename T::storage* __restrict__ y,
                      const float* __restrict__ gamma, const float* __restrict__ beta, const float* __restrict__ mean,
                      const float* __restrict__ invstd, int rows, NhwcShape s) {
    grid_dependency_wait();
    grid_dependency_launch();
    const NhwcThread me(s);
    if (!me.active) return;
    float a[V], b[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const int c = me.cv * V + j;
        a[j] = gamma[c] * invstd[c];
        b[j] = fmaf(-mean[c], a[j], beta[c]);
    }
    const int q0 = blockIdx.x * s.rows_per_block, q1 = min(rows, q0 + s.rows_per_block);
    const size_t col = static_cast<size_t>(me.cv) * V;
    for (int q = q0 + me.rl; q < q1; q += kUnroll * s.RL) {
        Vec<T, V> v[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (q + u * s.RL < q1) v[u].load(x + static_cast<size_t>(q + u * s.RL) * s.C + col);
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (q + u * s.RL < q1) {
#pragma unroll
                for (int j = 0; j < V; ++j) v[u].set(j, fmaf(a[j], v[u].get(j), b[j]));
                v[u].store(y + static_cast<size_t>(q + u * s.RL) * s.C + col);
            }
    }
}

// ------------------------------------------------------------------------------------ backward, pass 1
template <typename T, int V, bool WRITE_DX>
__global__ void __launch_bounds__(kThreads)
nhwc_bwd_reduce_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                       typename T::storage* __restrict__ dx, const float* __restrict__ gamma,
                       const float* __restrict__ mean, const float* __restrict__ invstd, int rows, NhwcShape s,
                       float2* __restrict__ partials) {
    __shared__ float s_dy[kThreads * V], s_dyxc[kThreads * V];
    grid_dependency_wait();
    grid_dependency_launch();
    const NhwcThread me(s);
    float acc_dy[V], acc_dyxc[V];
#pragma unroll
    for (int j = 0; j < V; ++j) acc_dy[j] = acc_dyxc[j] = 0.f;
    if (me.active) {
        float a[V], mu[V];
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const int c = me.cv * V + j;
            mu[j] = mean[c];
            a[j] = WRITE_DX ? gamma[c] * invstd[c] : 0.f;
        }
        const int q0 = blockIdx.x * s.rows_per_block, q1 = min(rows, q0 + s.rows_per_block);
        const size_t col = static_cast<size_t>(me.cv) * V;
        for (int q = q0 + me.rl; q < q1; q += kUnroll * s.RL) {
            Vec<T, V> vx[kUnroll], vg[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (q + u * s.RL < q1) {
                    const size_t off = static_cast<size_t>(q + u * s.RL) * s.C + col;
                    vx[u].load(x + off);
                    vg[u].load(dy + off);
                }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
                if (q + u * s.RL < q1) {
#pragma unroll
                    for (int j = 0; j < V; ++j) {
                        float g = vg[u].get(j);
                        acc_dy[j] += g;
                        acc_dyxc[j] = fmaf(g, vx[u].get(j) - mu[j], acc_dyxc[j]);
                        if (WRITE_DX) vg[u].set(j, a[j] * g);
                    }
                    if (WRITE_DX) vg[u].store(dx + static_cast<size_t>(q + u * s.RL) * s.C + col);
                }
        }
    }
#pragma unroll
    for (int j = 0; j < V; ++j) {
        s_dy[threadIdx.x * V + j] = acc_dy[j];
        s_dyxc[threadIdx.x * V + j] = acc_dyxc[j];
    }
    __syncthreads();
    for (int ch = threadIdx.x; ch < s.CW * V; ch += kThreads) {
        const int cvi = ch / V, j = ch - cvi * V;
        const int c = (blockIdx.y * s.CW + cvi) * V + j;
        if (c >= s.C) continue;
        float sa = 0.f, sb = 0.f;
        for (int rl = 0; rl < s.RL; ++rl) {
            const int t = rl * s.CW + cvi;
            sa += s_dy[t * V + j];
            sb += s_dyxc[t * V + j];
        }
        partials[static_cast<size_t>(blockIdx.x) * s.C + c] = make_float2(sa, sb);
    }
}

// ------------------------------------------------------------------------------------ backward, statistics terms
// dx = a dy - A - Q (x - mean) on the rows of the set; dy == NULL reads as zeros.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
nhwc_fixup_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                  typename T::storage* __restrict__ dx, const float* __restrict__ gamma, const float* __restrict__ mean,
                  const float* __restrict__ invstd, const float* __restrict__ dgamma, const float* __restrict__ dbeta,
                  float inv_s, RowSet set, NhwcShape s, unsigned* status) {
    grid_dependency_wait();
    grid_dependency_launch();
    const NhwcThread me(s);
    if (!me.active) return;
    FixCoef k[V];
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const int c = me.cv * V + j;
        k[j] = fix_coef(gamma[c], mean[c], invstd[c], dgamma[c], dbeta[c], inv_s);
    }
    const int q0 = blockIdx.x * s.rows_per_block, q1 = min(set.total, q0 + s.rows_per_block);
    const size_t col = static_cast<size_t>(me.cv) * V;
    for (int q = q0 + me.rl; q < q1; q += kUnroll * s.RL) {
        Vec<T, V> vx[kUnroll], vg[kUnroll];
        size_t off[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (q + u * s.RL < q1) {
                off[u] = static_cast<size_t>(set.row(q + u * s.RL, status)) * s.C + col;
                vx[u].load(x + off[u]);
                if (dy) vg[u].load(dy + off[u]);
            }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (q + u * s.RL < q1) {
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    float g = dy ? vg[u].get(j) : 0.f;
                    vg[u].set(j, fmaf(k[j].a, g, -k[j].A) - k[j].Q * (vx[u].get(j) - k[j].mu));
                }
                vg[u].store(dx + off[u]);
            }
    }
}

// ------------------------------------------------------------------------------------ small sampled sets
// When the sampled set is a few thousand rows (small patches, a couple of samples) one block per narrow
// strip of channels can visit all of it: the statistics then need no partials and no finalize launch, and
// in the backward the block that combines the strip's partial sums applies the statistics terms to the
// strip's sampled elements right away.  The grid is (1, strips); a block is CW (1 or 2) channel-vectors
// wide - 32 bytes of every sampled row - and kThreads / CW row-lanes deep.
constexpr int kNhwcDirectUnroll = 8;  // rows a thread keeps in flight

// Sum over the row-lanes of a block, in a fixed order: lanes of a warp by a shuffle tree (a warp holds
// 32 / CW row-lanes of each channel-vector, CW a power of two), then the warps through shared memory.
// The totals land in shared memory: s_out[cvi * NV + i] for value i of channel-vector cvi of the block.
template <int NV>
__device__ __forceinline__ void nhwc_block_sum(float (&val)[NV], int CW, float* s_warp, float* s_out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
#pragma unroll
    for (int i = 0; i < NV; ++i)
        for (int d = CW; d < 32; d <<= 1) val[i] += __shfl_xor_sync(0xffffffffu, val[i], d);
    if (lane < CW) {
#pragma unroll
        for (int i = 0; i < NV; ++i) s_warp[(warp * 2 + lane) * NV + i] = val[i];
    }
    __syncthreads();
    for (int e = threadIdx.x; e < CW * NV; e += kThreads) {
        const int cvi = e / NV, i = e - cvi * NV;
        float tot = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) tot += s_warp[(w * 2 + cvi) * NV + i];
        s_out[e] = tot;
    }
    __syncthreads();
}

// mean and invstd of the block's channels straight from the sampled rows.  Sums are shifted by the value of
// the first sampled row (one pivot per channel for the whole block, so the lanes' sums simply add).
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
nhwc_direct_moments_kernel(const typename T::storage* __restrict__ x, RowSet set, NhwcShape s, float eps,
                           float* __restrict__ mean, float* __restrict__ invstd, unsigned* status) {
    constexpr int U = kNhwcDirectUnroll;
    __shared__ float s_warp[(kThreads / 32) * 2 * 2 * V];
    __shared__ float s_tot[2 * 2 * V];
    grid_dependency_wait();
    grid_dependency_launch();
    const NhwcThread me(s);
    float K[V], sums[2 * V];
#pragma unroll
    for (int j = 0; j < V; ++j) K[j] = sums[j] = sums[V + j] = 0.f;
    if (me.active) {
        const typename T::storage* xp = x + static_cast<size_t>(me.cv) * V;
        Vec<T, V> first;
        first.load(xp + static_cast<size_t>(set.row(0, status)) * s.C);
#pragma unroll
        for (int j = 0; j < V; ++j) K[j] = first.get(j);
        for (int q = me.rl; q < set.total; q += U * s.RL) {
            Vec<T, V> v[U];
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (q + u * s.RL < set.total) v[u].load(xp + static_cast<size_t>(set.row(q + u * s.RL, status)) * s.C);
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (q + u * s.RL < set.total) {
#pragma unroll
                    for (int j = 0; j < V; ++j) {
                        const float d = v[u].get(j) - K[j];
                        sums[j] += d;
                        sums[V + j] = fmaf(d, d, sums[V + j]);
                    }
                }
        }
    }
    nhwc_block_sum<2 * V>(sums, s.CW, s_warp, s_tot);
    // thread (rl == 0, cvi) finishes the V channels of its vector; it holds their pivots
    if (me.active && me.rl == 0) {
        const int cvi = threadIdx.x % s.CW;
        const float n = static_cast<float>(set.total);
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float s1 = s_tot[cvi * 2 * V + j], s2 = s_tot[cvi * 2 * V + V + j];
            const float m2 = fmaxf(s2 - s1 * s1 / n, 0.f);
            mean[me.cv * V + j] = K[j] + s1 / n;
            invstd[me.cv * V + j] = 1.0f / sqrtf(m2 / n + eps);
        }
    }
}

// Backward for a small sampled set: the block adds up the partial sums that pass 1 left for its channels
// (every block of pass 1 wrote one per channel), publishes dgamma / dbeta, and rewrites the gradient of the
// strip's sampled elements with the statistics terms.  dy == NULL reads as zeros; dx == NULL skips the rewrite.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
nhwc_direct_finalize_fixup_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                                  typename T::storage* __restrict__ dx, const float* __restrict__ gamma,
                                  const float* __restrict__ mean, const float* __restrict__ invstd,
                                  const float2* __restrict__ partials, int entries,
                                  const float2* __restrict__ partials_v, int entries_v, float inv_s, RowSet set,
                                  NhwcShape s, float* __restrict__ dgamma, float* __restrict__ dbeta, unsigned* status) {
    constexpr int U = kNhwcDirectUnroll;
    __shared__ float2 s_part[kThreads];
    __shared__ float2 s_grad[2 * V];
    grid_dependency_wait();
    grid_dependency_launch();
    const NhwcThread me(s);
    // partial sums: thread t adds the entries el, el + lanes, ... of channel ch of the strip (neighbouring threads
    // read neighbouring channels of one entry), then thread ch adds the lanes' results in lane order
    const int nch = s.CW * V, lanes = kThreads / nch;
    const int ch = threadIdx.x % nch, el = threadIdx.x / nch;
    const int c_of_ch = blockIdx.y * nch + ch;
    float sa = 0.f, sb = 0.f;
    if (el < lanes && c_of_ch < s.C) {
        for (int pass = 0; pass < 2; ++pass) {
            const float2* src = pass ? partials_v : partials;
            const int n = pass ? entries_v : entries;
            if (!src) continue;
            for (int e = el; e < n; e += U * lanes) {  // batches of U loads in flight, added in entry order
                float2 v[U];
#pragma unroll
                for (int u = 0; u < U; ++u)
                    v[u] = e + u * lanes < n ? src[static_cast<size_t>(e + u * lanes) * s.C + c_of_ch] : make_float2(0.f, 0.f);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    sa += v[u].x;
                    sb += v[u].y;
                }
            }
        }
    }
    s_part[threadIdx.x] = make_float2(sa, sb);
    __syncthreads();
    if (threadIdx.x < nch && c_of_ch < s.C) {
        float ta = 0.f, tb = 0.f;
        for (int l = 0; l < lanes; ++l) {
            ta += s_part[l * nch + threadIdx.x].x;
            tb += s_part[l * nch + threadIdx.x].y;
        }
        tb *= invstd[c_of_ch];
        dbeta[c_of_ch] = ta;
        dgamma[c_of_ch] = tb;
        s_grad[threadIdx.x] = make_float2(tb, ta);  // (dgamma, dbeta)
    }
    __syncthreads();
    if (!dx || !me.active) return;
    FixCoef k[V];
    const int cvi = threadIdx.x % s.CW;
#pragma unroll
    for (int j = 0; j < V; ++j) {
        const int c = me.cv * V + j;
        const float2 g = s_grad[cvi * V + j];
        k[j] = fix_coef(gamma[c], mean[c], invstd[c], g.x, g.y, inv_s);
    }
    const size_t col = static_cast<size_t>(me.cv) * V;
    for (int q = me.rl; q < set.total; q += U * s.RL) {
        Vec<T, V> vx[U], vg[U];
        size_t off[U];
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (q + u * s.RL < set.total) {
                off[u] = static_cast<size_t>(set.row(q + u * s.RL, status)) * s.C + col;
                vx[u].load(x + off[u]);
                if (dy) vg[u].load(dy + off[u]);
            }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (q + u * s.RL < set.total) {
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    const float g = dy ? vg[u].get(j) : 0.f;
                    vg[u].set(j, fmaf(k[j].a, g, -k[j].A) - k[j].Q * (vx[u].get(j) - k[j].mu));
                }
                vg[u].store(dx + off[u]);
            }
    }
}

// ------------------------------------------------------------------------------------ combining the blocks' partials
// Every block of a channels-last pass leaves one partial per channel: partial[block*C + c].  Here lane l
// of a warp owns channel 32*blockIdx.x + l (neighbouring lanes read neighbouring addresses) and the 32
// warps of a 1024-thread block share the entries, each loading a batch before it adds; the warps' results
// meet in shared memory and are combined in warp order.
constexpr int kFinalizeThreads = 1024;
constexpr int kFinalizeWarps = kFinalizeThreads / 32;

__global__ void __launch_bounds__(kFinalizeThreads)
nhwc_finalize_stats_kernel(const float4* __restrict__ partials, int entries, int C, float inv_s, float eps,
                           float* __restrict__ mean, float* __restrict__ invstd) {
    __shared__ float s_cnt[kFinalizeThreads], s_mean[kFinalizeThreads], s_m2[kFinalizeThreads];
    grid_dependency_wait();
    grid_dependency_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = blockIdx.x * 32 + lane;
    Moments acc = {0.f, 0.f, 0.f};
    if (c < C) {
        constexpr int kBatch = 4;
        for (int e = warp; e < entries; e += kBatch * kFinalizeWarps) {
            float4 v[kBatch];
#pragma unroll
            for (int u = 0; u < kBatch; ++u)
                v[u] = e + u * kFinalizeWarps < entries ? partials[static_cast<size_t>(e + u * kFinalizeWarps) * C + c]
                                                        : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int u = 0; u < kBatch; ++u) acc = merge(acc, Moments{v[u].x, v[u].y, v[u].z});
        }
    }
    s_cnt[threadIdx.x] = acc.cnt;
    s_mean[threadIdx.x] = acc.mean;
    s_m2[threadIdx.x] = acc.m2;
    __syncthreads();
    if (warp == 0 && c < C) {
        Moments tot = {0.f, 0.f, 0.f};
        for (int w = 0; w < kFinalizeWarps; ++w)
            tot = merge(tot, Moments{s_cnt[w * 32 + lane], s_mean[w * 32 + lane], s_m2[w * 32 + lane]});
        mean[c] = tot.mean;
        invstd[c] = 1.0f / sqrtf(tot.m2 * inv_s + eps);
    }
}

__global__ void __launch_bounds__(kFinalizeThreads)
nhwc_finalize_bwd_kernel(const float2* __restrict__ partials, int entries, const float2* __restrict__ partials_v,
                         int entries_v, int C, const float* __restrict__ invstd, float* __restrict__ dgamma,
                         float* __restrict__ dbeta) {
    __shared__ float s_a[kFinalizeThreads], s_b[kFinalizeThreads];
    grid_dependency_wait();
    grid_dependency_launch();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int c = blockIdx.x * 32 + lane;
    float sa = 0.f, sb = 0.f;
    if (c < C) {
        constexpr int kBatch = 4;
        for (int pass = 0; pass < 2; ++pass) {
            const float2* src = pass ? partials_v : partials;
            const int n = pass ? entries_v : entries;
            if (!src) continue;
            for (int e = warp; e < n; e += kBatch * kFinalizeWarps) {
                float2 v[kBatch];
#pragma unroll
                for (int u = 0; u < kBatch; ++u)
                    v[u] = e + u * kFinalizeWarps < n ? src[static_cast<size_t>(e + u * kFinalizeWarps) * C + c]
                                                      : make_float2(0.f, 0.f);
#pragma unroll
                for (int u = 0; u < kBatch; ++u) {
                    sa += v[u].x;
                    sb += v[u].y;
                }
            }
        }
    }
    s_a[threadIdx.x] = sa;
    s_b[threadIdx.x] = sb;
    __syncthreads();
    if (warp == 0 && c < C) {
        float ta = 0.f, tb = 0.f;
        for (int w = 0; w < kFinalizeWarps; ++w) {
            ta += s_a[w * 32 + lane];
            tb += s_b[w * 32 + lane];
        }
        dbeta[c] = ta;
        dgamma[c] = tb * invstd[c];
    }
}

}  // namespace bns

// Device code of the BN-sampling library (sm_100a).
//
// Data layout.  A dense NCHW tensor is seen as N rows of P = C*H*W contiguous "positions"; the
// channel of position p is p / (H*W).  The streaming kernels ("col_*") give every thread V
// consecutive positions (V elements = up to 16 bytes) and let it walk down the rows n of its chunk:
// the per-channel parameters of its V positions are looked up once, before the loop, every access
// is a full-width coalesced vector, and per-channel sums are kept per position in registers, so the
// inner loop holds no index arithmetic, no shuffles and no shared memory.  Only after the loop are
// the per-position sums folded into per-channel partials (one block-level pass through shared
// memory), which a small "finalize" kernel (one warp per channel) combines in a fixed order.
//
// Feature Sampling uses the same scheme on a compacted position space: a sample row then has only
// C*ph*pw positions (the patch elements of every map), thread j owns patch element j % (ph*pw) of
// channel j / (ph*pw), and consecutive threads touch consecutive patch columns, rows and channels,
// i.e. neighbouring addresses.
//
// Every kernel starts with a programmatic-dependent-launch wait, so that with the launch attribute
// set its blocks may be scheduled while the previous kernel of the stream drains; nothing is read or
// written before that wait.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bns {

constexpr int kThreads = 256;  // threads per block of every streaming kernel
constexpr int kUnroll = 4;     // rows in flight per thread

// Programmatic dependent launch: wait until the preceding kernel of the stream has completed and
// its writes are visible (a no-op when the launch did not ask for early scheduling).
__device__ __forceinline__ void grid_dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
// Allow the next kernel of the stream to be scheduled once every block of this one got here.
__device__ __forceinline__ void grid_dependency_launch() { asm volatile("griddepcontrol.launch_dependents;"); }

// ------------------------------------------------------------------------------------ row order
// Row chunks are interleaved: chunk ck of nchunks visits "virtual rows" ck, ck+nchunks, ck+2 nchunks, ...
// so all blocks of a launch move through the tensor together and virtual row v is visited at about
// the same time by every block.  RowOrder maps the virtual row to the sample it stands for, which
// lets a kernel visit first the rows that the previous kernel left in L2, or leave for last the rows
// that the next kernel will want there.  The order only permutes independent rows.
struct RowOrder {
    enum { kIdentity = 0, kRangeFirst = 1, kRangeLast = 2, kReversed = 3 };
    int mode, rows, begin, count;  // [begin, begin+count): the range moved to the front or to the back
    __device__ __forceinline__ int operator()(int v) const {
        switch (mode) {
        case kRangeFirst: return v < count ? begin + v : (v - count < begin ? v - count : v);
        case kRangeLast: return v < begin ? v : (v < rows - count ? v + count : begin + v - (rows - count));
        case kReversed: return rows - 1 - v;
        default: return v;
        }
    }
};

// ------------------------------------------------------------------------------------ element types
struct F32 {
    using storage = float;
};
struct BF16 {
    using storage = unsigned short;
};

template <typename T>
__device__ __forceinline__ float to_float(typename T::storage v);
template <>
__device__ __forceinline__ float to_float<F32>(float v) {
    return v;
}
template <>
__device__ __forceinline__ float to_float<BF16>(unsigned short v) {
    return __uint_as_float(static_cast<unsigned>(v) << 16);
}
template <typename T>
__device__ __forceinline__ typename T::storage from_float(float v);
template <>
__device__ __forceinline__ float from_float<F32>(float v) {
    return v;
}
template <>
__device__ __forceinline__ unsigned short from_float<BF16>(float v) {
    return __bfloat16_as_ushort(__float2bfloat16_rn(v));  // round to nearest even
}

template <int BYTES>
struct RawWord;
template <>
struct RawWord<2> {
    using type = unsigned short;
};
template <>
struct RawWord<4> {
    using type = unsigned;
};
template <>
struct RawWord<8> {
    using type = uint2;
};
template <>
struct RawWord<16> {
    using type = uint4;
};

// V consecutive elements moved as one machine word of 2..16 bytes.
template <typename T, int V>
struct Vec {
    using S = typename T::storage;
    using raw_t = typename RawWord<sizeof(S) * V>::type;
    raw_t raw;
    __device__ __forceinline__ void load(const S* p) { raw = *reinterpret_cast<const raw_t*>(p); }
    __device__ __forceinline__ void store(S* p) const { *reinterpret_cast<raw_t*>(p) = raw; }
    __device__ __forceinline__ float get(int j) const { return to_float<T>(reinterpret_cast<const S*>(&raw)[j]); }
    __device__ __forceinline__ void set(int j, float v) { reinterpret_cast<S*>(&raw)[j] = from_float<T>(v); }
    // whole-vector conversion; the bf16 case works on 32-bit pairs (one shift or mask per element on the
    // way in, one cvt.rn.bf16x2.f32 per pair on the way out)
    __device__ __forceinline__ void unpack(float (&f)[V]) const {
        if constexpr (sizeof(S) == 2 && V >= 2) {
            const unsigned* w = reinterpret_cast<const unsigned*>(&raw);
#pragma unroll
            for (int q = 0; q < V / 2; ++q) {
                f[2 * q] = __uint_as_float(w[q] << 16);
                f[2 * q + 1] = __uint_as_float(w[q] & 0xffff0000u);
            }
        } else {
#pragma unroll
            for (int j = 0; j < V; ++j) f[j] = get(j);
        }
    }
    __device__ __forceinline__ void pack(const float (&f)[V]) {
        if constexpr (sizeof(S) == 2 && V >= 2) {
            unsigned* w = reinterpret_cast<unsigned*>(&raw);
#pragma unroll
            for (int q = 0; q < V / 2; ++q) {
                __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * q], f[2 * q + 1]);  // low half = first argument
                w[q] = *reinterpret_cast<unsigned*>(&h);
            }
        } else {
#pragma unroll
            for (int j = 0; j < V; ++j) set(j, f[j]);
        }
    }
};

// Two fp32 values in one 64-bit register pair, for the packed fp32x2 arithmetic of sm_100 (each half is
// an ordinary round-to-nearest fp32 operation, so results equal the scalar ones bit for bit).
using pair_t = unsigned long long;
__device__ __forceinline__ pair_t make_pair(float lo, float hi) {
    pair_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void split_pair(pair_t v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ pair_t add2(pair_t a, pair_t b) {
    pair_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ pair_t mul2(pair_t a, pair_t b) {
    pair_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ pair_t fma2(pair_t a, pair_t b, pair_t c) {
    pair_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Elements 2q and 2q+1 of a vector as a pair, and back (bf16: one 32-bit word holds both).
template <typename T, int V>
__device__ __forceinline__ pair_t vec_pair(const Vec<T, V>& v, int q) {
    if constexpr (sizeof(typename T::storage) == 2) {
        const unsigned w = reinterpret_cast<const unsigned*>(&v.raw)[q];
        return make_pair(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
    } else {
        const float* f = reinterpret_cast<const float*>(&v.raw);
        return make_pair(f[2 * q], f[2 * q + 1]);
    }
}
template <typename T, int V>
__device__ __forceinline__ void set_vec_pair(Vec<T, V>& v, int q, pair_t p) {
    float lo, hi;
    split_pair(p, lo, hi);
    if constexpr (sizeof(typename T::storage) == 2) {
        __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);  // low half = first argument
        reinterpret_cast<unsigned*>(&v.raw)[q] = *reinterpret_cast<unsigned*>(&h);
    } else {
        float* f = reinterpret_cast<float*>(&v.raw);
        f[2 * q] = lo;
        f[2 * q + 1] = hi;
    }
}

// Channels of the V positions p .. p+V-1 (HW may be smaller than V).
template <int V>
__device__ __forceinline__ void position_channels(unsigned p, int HW, int (&c)[V]) {
    int c0 = static_cast<int>(p / static_cast<unsigned>(HW));
    int r = static_cast<int>(p - static_cast<unsigned>(c0) * static_cast<unsigned>(HW));
#pragma unroll
    for (int j = 0; j < V; ++j) {
        c[j] = c0;
        if (++r == HW) {
            r = 0;
            ++c0;
        }
    }
}

// When a feature map holds at least V positions, the V positions of a thread meet at most two channels:
// c0 for positions j < jb and c0 + 1 from jb on (jb = V when the thread stays inside one channel).
struct TwoChannels {
    int c0, c1, jb;
    __device__ __forceinline__ TwoChannels(unsigned p, int HW, int V) {
        c0 = static_cast<int>(p / static_cast<unsigned>(HW));
        const int r = static_cast<int>(p - static_cast<unsigned>(c0) * static_cast<unsigned>(HW));
        jb = min(V, HW - r);
        c1 = jb < V ? c0 + 1 : c0;
    }
    __device__ __forceinline__ float pick(int j, float lo, float hi) const { return j < jb ? lo : hi; }
};

// ------------------------------------------------------------------------------------ moments
// (count, mean, sum of squared deviations) of a set; merge() is the pairwise update of Chan et al.
struct Moments {
    float cnt, mean, m2;
};

__device__ __forceinline__ Moments merge(Moments a, Moments b) {
    float n = a.cnt + b.cnt;
    if (n == 0.f) return a;
    float d = b.mean - a.mean;
    float f = b.cnt / n;
    Moments r;
    r.cnt = n;
    r.mean = a.mean + d * f;
    r.m2 = a.m2 + b.m2 + d * d * a.cnt * f;
    return r;
}

__device__ __forceinline__ Moments shuffle_down(Moments m, int delta) {
    Moments r;
    r.cnt = __shfl_down_sync(0xffffffffu, m.cnt, delta);
    r.mean = __shfl_down_sync(0xffffffffu, m.mean, delta);
    r.m2 = __shfl_down_sync(0xffffffffu, m.m2, delta);
    return r;
}

__device__ __forceinline__ Moments warp_merge(Moments m) {
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) m = merge(m, shuffle_down(m, d));
    return m;  // complete in lane 0
}

// Moments of one position from sums shifted by a pivot K that is itself one of the values:
// sum1 = sum(x-K), sum2 = sum((x-K)^2) over cnt values.
__device__ __forceinline__ Moments from_shifted_sums(float cnt, float K, float sum1, float sum2) {
    Moments m;
    m.cnt = cnt;
    if (cnt == 0.f) {
        m.mean = 0.f;
        m.m2 = 0.f;
        return m;
    }
    float d = sum1 / cnt;
    m.mean = K + d;
    m.m2 = fmaxf(sum2 - sum1 * d, 0.f);
    return m;
}

// Where a block's tile of positions [p0, p0+TP) meets the channels: slot j is channel c_first + j.
struct TileChannels {
    unsigned p0, pend;
    int c_first, nslots;
    __device__ __forceinline__ TileChannels(unsigned tile, unsigned TP, unsigned P, int HW) {
        p0 = tile * TP;
        pend = min(p0 + TP, P);
        c_first = static_cast<int>(p0 / static_cast<unsigned>(HW));
        nslots = static_cast<int>((pend - 1) / static_cast<unsigned>(HW)) - c_first + 1;
    }
    // positions of slot j, relative to p0
    __device__ __forceinline__ void range(int slot, int HW, unsigned& lo, unsigned& hi) const {
        unsigned cb = static_cast<unsigned>(c_first + slot) * static_cast<unsigned>(HW);
        lo = max(cb, p0) - p0;
        hi = min(cb + static_cast<unsigned>(HW), pend) - p0;
    }
};

// ------------------------------------------------------------------------------------ partials and how they are combined
// How the partials of one pass are indexed: partial[(chunk*tiles + tile)*max_slots + slot], where
// tile t covers positions [t*TP, (t+1)*TP) of a row and slot = channel - first channel of the tile.
// The per-(chunk, channel) layout of the patch kernels is the case TP = HW, tiles = C, max_slots = 1.
struct PartialLayout {
    int nchunks;
    unsigned tiles, TP;
    int max_slots;
    // partials that channel c receives: one per (row chunk, tile that meets the channel)
    __device__ __forceinline__ int entries(int c, int HW, unsigned& t_lo, int& nt) const {
        const unsigned pb = static_cast<unsigned>(c) * HW;
        t_lo = pb / TP;
        nt = static_cast<int>((pb + HW - 1) / TP - t_lo + 1);
        return nchunks * nt;
    }
};

// Eq. 8: the moving averages of E and Var that validation uses, updated by whichever thread finishes a
// channel's statistics (X_ma = X at the first iteration, alpha X + (1 - alpha) X_ma afterwards).  Inactive
// when mean_ma is NULL.
struct MovingAverage {
    float alpha;
    int first;
    float* mean_ma;
    float* var_ma;
    __device__ __forceinline__ void update(int c, float mean, float var) const {
        if (!mean_ma) return;
        mean_ma[c] = first ? mean : alpha * mean + (1.0f - alpha) * mean_ma[c];
        var_ma[c] = first ? var : alpha * var + (1.0f - alpha) * var_ma[c];
    }
};

// Statistics: where the partial moments are and where the finished mean / invstd go.
struct StatsSink {
    float4* partials;
    PartialLayout L;
    float inv_s, eps;
    float* mean;
    float* invstd;
    MovingAverage ma;
};

// All partial moments of channel c, merged in a fixed order by one warp; mean / invstd written by lane 0.
__device__ __forceinline__ void warp_finish_stats(const StatsSink& S, int c, int HW, int lane) {
    unsigned t_lo;
    int nt;
    const int entries = S.L.entries(c, HW, t_lo, nt);
    Moments acc = {0.f, 0.f, 0.f};
    for (int e = lane; e < entries; e += 32) {
        int ck = e / nt;
        unsigned t = t_lo + static_cast<unsigned>(e - ck * nt);
        int slot = c - static_cast<int>((t * S.L.TP) / static_cast<unsigned>(HW));
        float4 v = S.partials[(static_cast<size_t>(ck) * S.L.tiles + t) * S.L.max_slots + slot];
        acc = merge(acc, Moments{v.x, v.y, v.z});
    }
    acc = warp_merge(acc);
    if (lane == 0) {
        S.mean[c] = acc.mean;
        S.invstd[c] = 1.0f / sqrtf(acc.m2 * S.inv_s + S.eps);
        S.ma.update(c, acc.mean, acc.m2 * S.inv_s);
    }
}

// Backward sums: partial (sum dy, sum dy (x - mean)) pairs of the real tensor and, when present, of the
// virtual samples; both feed the same channel.
struct GradSink {
    float2* partials;
    PartialLayout L;
    float2* partials_v;  // NULL when no virtual gradient takes part
    PartialLayout Lv;
    const float* invstd;
    float* dgamma;
    float* dbeta;
};

// All partial sums of channel c, added in a fixed order by one warp; lane 0 returns (dgamma, dbeta).
__device__ __forceinline__ float2 warp_sum_grads(const GradSink& G, int c, int HW, int lane) {
    float sum_dy = 0.f, sum_dyxc = 0.f;
    for (int pass = 0; pass < 2; ++pass) {
        const float2* src = pass ? G.partials_v : G.partials;
        if (!src) continue;
        const PartialLayout& Q = pass ? G.Lv : G.L;
        unsigned t_lo;
        int nt;
        const int entries = Q.entries(c, HW, t_lo, nt);
        for (int e = lane; e < entries; e += 32) {
            int ck = e / nt;
            unsigned t = t_lo + static_cast<unsigned>(e - ck * nt);
            int slot = c - static_cast<int>((t * Q.TP) / static_cast<unsigned>(HW));
            float2 v = src[(static_cast<size_t>(ck) * Q.tiles + t) * Q.max_slots + slot];
            sum_dy += v.x;
            sum_dyxc += v.y;
        }
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        sum_dy += __shfl_down_sync(0xffffffffu, sum_dy, d);
        sum_dyxc += __shfl_down_sync(0xffffffffu, sum_dyxc, d);
    }
    return make_float2(sum_dyxc * G.invstd[c], sum_dy);
}

__device__ __forceinline__ void warp_finish_grads(const GradSink& G, int c, int HW, int lane) {
    const float2 g = warp_sum_grads(G, c, HW, lane);
    if (lane == 0) {
        G.dgamma[c] = g.x;
        G.dbeta[c] = g.y;
    }
}

// The fix-up kernels can finish the sums themselves instead of reading dgamma / dbeta from a finalize
// launch: every block adds up, in the same fixed order, the partials of the (few) channels its tile
// meets, and the one block that holds a channel's first position in the first row chunk publishes them.
// s_grad[slot] = (dgamma, dbeta) of channel c_first + slot; ends with a block barrier.
constexpr int kFoldSlots = 32;  // most channels per tile for which a fix-up kernel finishes the sums itself

__device__ __forceinline__ void block_finish_grads(const GradSink& G, int c_first, int nslots, int HW, bool first_chunk,
                                                   unsigned tile, unsigned positions_per_tile, int positions_per_channel,
                                                   float2* s_grad) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int slot = warp; slot < nslots; slot += kThreads / 32) {
        const int c = c_first + slot;
        const float2 g = warp_sum_grads(G, c, HW, lane);
        if (lane == 0) {
            s_grad[slot] = g;
            const unsigned home = static_cast<unsigned>(c) * static_cast<unsigned>(positions_per_channel) / positions_per_tile;
            if (first_chunk && home == tile) {
                G.dgamma[c] = g.x;
                G.dbeta[c] = g.y;
            }
        }
    }
    __syncthreads();
}

// Folds the per-position moments of a block's tile (shared memory, one entry per position, every
// position holding `cnt` values) into one partial per channel the tile meets.  The channel mean is the
// plain average of the position means and M2 = sum(M2_q) + cnt * sum((mean_q - mean)^2): two passes of
// plain sums, no divisions per element.  `span` is the number of positions per channel.
__device__ __forceinline__ void fold_moments(const float* s_mean, const float* s_m2, float cnt, const TileChannels& tc,
                                             int span, float4* out) {
    if (span >= 32) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int slot = warp; slot < tc.nslots; slot += kThreads / 32) {
            unsigned lo, hi;
            tc.range(slot, span, lo, hi);
            float sum = 0.f;
            for (unsigned q = lo + lane; q < hi; q += 32) sum += s_mean[q];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, d);
            const float len = static_cast<float>(hi - lo);
            const float mu = sum / len;
            float dev = 0.f, m2 = 0.f;
            for (unsigned q = lo + lane; q < hi; q += 32) {
                float d = s_mean[q] - mu;
                dev = fmaf(d, d, dev);
                m2 += s_m2[q];
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                dev += __shfl_xor_sync(0xffffffffu, dev, d);
                m2 += __shfl_xor_sync(0xffffffffu, m2, d);
            }
            if (lane == 0) out[slot] = make_float4(cnt * len, mu, fmaf(cnt, dev, m2), 0.f);
        }
    } else {
        // fewer positions per channel than a warp has lanes: one thread per channel
        for (int slot = threadIdx.x; slot < tc.nslots; slot += kThreads) {
            unsigned lo, hi;
            tc.range(slot, span, lo, hi);
            float sum = 0.f;
            for (unsigned q = lo; q < hi; ++q) sum += s_mean[q];
            const float len = static_cast<float>(hi - lo);
            const float mu = sum / len;
            float dev = 0.f, m2 = 0.f;
            for (unsigned q = lo; q < hi; ++q) {
                float d = s_mean[q] - mu;
                dev = fmaf(d, d, dev);
                m2 += s_m2[q];
            }
            out[slot] = make_float4(cnt * len, mu, fmaf(cnt, dev, m2), 0.f);
        }
    }
}

// The same for plain sums (backward): one (sum dy, sum dy (x - mean)) pair per channel the tile meets.
__device__ __forceinline__ void fold_sums(const float* s_a, const float* s_b, const TileChannels& tc, int span,
                                          float2* out) {
    if (span >= 32) {
        const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
        for (int slot = warp; slot < tc.nslots; slot += kThreads / 32) {
            unsigned lo, hi;
            tc.range(slot, span, lo, hi);
            float sa = 0.f, sb = 0.f;
            for (unsigned q = lo + lane; q < hi; q += 32) {
                sa += s_a[q];
                sb += s_b[q];
            }
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) {
                sa += __shfl_down_sync(0xffffffffu, sa, d);
                sb += __shfl_down_sync(0xffffffffu, sb, d);
            }
            if (lane == 0) out[slot] = make_float2(sa, sb);
        }
    } else {
        for (int slot = threadIdx.x; slot < tc.nslots; slot += kThreads) {
            unsigned lo, hi;
            tc.range(slot, span, lo, hi);
            float sa = 0.f, sb = 0.f;
            for (unsigned q = lo; q < hi; ++q) {
                sa += s_a[q];
                sb += s_b[q];
            }
            out[slot] = make_float2(sa, sb);
        }
    }
}

// ------------------------------------------------------------------------------------ statistics over whole samples
// Partial moments of x[list, :] per (row chunk, tile, channel slot).  `list` (device) holds the
// sample indices or is NULL for the contiguous range begin .. begin+count-1.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
col_moments_kernel(const typename T::storage* __restrict__ x, const int* __restrict__ list, int begin, int count,
                   int nchunks, unsigned tiles, int HW, unsigned P, StatsSink S) {
    constexpr unsigned TP = kThreads * V;
    __shared__ float s_mean[TP];
    __shared__ float s_m2[TP];
    grid_dependency_wait();
    grid_dependency_launch();
    const unsigned tile = blockIdx.x % tiles;
    const int ck = static_cast<int>(blockIdx.x / tiles);
    const unsigned p = (tile * kThreads + threadIdx.x) * V;
    const float cnt = static_cast<float>((count - ck + nchunks - 1) / nchunks);  // rows of this chunk
    float K[V], s1[V], s2[V];
#pragma unroll
    for (int j = 0; j < V; ++j) K[j] = s1[j] = s2[j] = 0.f;
    if (p < P) {
        const typename T::storage* xp = x + p;
        {   // pivot: the first value of every position (its own deviation is zero)
            int n = list ? list[ck] : begin + ck;
            Vec<T, V> v;
            v.load(xp + static_cast<size_t>(n) * P);
#pragma unroll
            for (int j = 0; j < V; ++j) K[j] = v.get(j);
        }
        int i = ck + nchunks;
        for (; i + (kUnroll - 1) * nchunks < count; i += kUnroll * nchunks) {
            Vec<T, V> v[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                int n = list ? list[i + u * nchunks] : begin + i + u * nchunks;
                v[u].load(xp + static_cast<size_t>(n) * P);
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u)
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    float d = v[u].get(j) - K[j];
                    s1[j] += d;
                    s2[j] = fmaf(d, d, s2[j]);
                }
        }
        for (; i < count; i += nchunks) {
            int n = list ? list[i] : begin + i;
            Vec<T, V> v;
            v.load(xp + static_cast<size_t>(n) * P);
#pragma unroll
            for (int j = 0; j < V; ++j) {
                float d = v.get(j) - K[j];
                s1[j] += d;
                s2[j] = fmaf(d, d, s2[j]);
            }
        }
    }
#pragma unroll
    for (int j = 0; j < V; ++j) {
        Moments m = from_shifted_sums(cnt, K[j], s1[j], s2[j]);
        s_mean[threadIdx.x * V + j] = m.mean;
        s_m2[threadIdx.x * V + j] = m.m2;
    }
    __syncthreads();
    fold_moments(s_mean, s_m2, cnt, TileChannels(tile, TP, P, HW), HW,
                 S.partials + (static_cast<size_t>(ck) * tiles + tile) * S.L.max_slots);
}

// ------------------------------------------------------------------------------------ statistics over patches
// Patch location of map (n, c): one pair for the layer, one per sample or one per map.  Pairs read
// from device memory are clamped into range; an out-of-range pair raises a flag in `status`.
struct PatchRule {
    int ph, pw;
    int oh, ow;          // SHARED location (validated on the host)
    const int* offsets;  // device pairs or NULL for SHARED
    int stride_n, stride_c;
};

__device__ __forceinline__ void patch_origin(const PatchRule& r, int n, int c, int H, int W, unsigned* status, int& oh,
                                             int& ow) {
    if (!r.offsets) {
        oh = r.oh;
        ow = r.ow;
        return;
    }
    size_t e = static_cast<size_t>(n) * r.stride_n + static_cast<size_t>(c) * r.stride_c;
    int2 o = reinterpret_cast<const int2*>(r.offsets)[e];
    oh = min(max(o.x, 0), H - r.ph);
    ow = min(max(o.y, 0), W - r.pw);
    if ((oh != o.x || ow != o.y) && status) atomicOr(status, 1u);
}

// A thread of the patch kernels owns compact position j of every sample row: patch element
// e = j % (ph*pw) (row e / pw, column e % pw of the patch) of channel c = j / (ph*pw).
struct PatchThread {
    int c, row, col;
    size_t plane;  // c*H*W + row*W + col: offset inside a sample row, before the patch origin is added
    __device__ __forceinline__ PatchThread(unsigned j, const PatchRule& r, int H, int W) {
        const int PP = r.ph * r.pw;
        c = static_cast<int>(j / static_cast<unsigned>(PP));
        const int e = static_cast<int>(j - static_cast<unsigned>(c) * PP);
        row = e / r.pw;
        col = e - row * r.pw;
        plane = static_cast<size_t>(c) * H * W + static_cast<size_t>(row) * W + col;
    }
    // element offset of this thread's patch element in sample n
    __device__ __forceinline__ size_t at(const PatchRule& r, int n, size_t P, int H, int W, unsigned* status) const {
        int oh, ow;
        patch_origin(r, n, c, H, W, status, oh, ow);
        return static_cast<size_t>(n) * P + plane + static_cast<size_t>(oh) * W + ow;
    }
};

// Partial moments of the patch elements per (sample chunk, tile of compact positions, channel slot).
template <typename T>
__global__ void __launch_bounds__(kThreads)
patch_moments_kernel(const typename T::storage* __restrict__ x, PatchRule rule, int N, int C, int H, int W, int nchunks,
                     unsigned tiles, StatsSink S, unsigned* status) {
    __shared__ float s_mean[kThreads];
    __shared__ float s_m2[kThreads];
    grid_dependency_wait();
    grid_dependency_launch();
    const unsigned tile = blockIdx.x % tiles;
    const int ck = static_cast<int>(blockIdx.x / tiles);
    const int PP = rule.ph * rule.pw;
    const unsigned Pc = static_cast<unsigned>(C) * PP;  // compact positions per sample
    const unsigned j = tile * kThreads + threadIdx.x;
    const size_t P = static_cast<size_t>(C) * H * W;
    const float cnt = static_cast<float>((N - ck + nchunks - 1) / nchunks);  // samples of this chunk
    float K = 0.f, s1 = 0.f, s2 = 0.f;
    if (j < Pc) {
        const PatchThread me(j, rule, H, W);
        K = to_float<T>(x[me.at(rule, ck, P, H, W, status)]);  // pivot: the first value
        int n = ck + nchunks;
        for (; n + (kUnroll - 1) * nchunks < N; n += kUnroll * nchunks) {
            float v[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) v[u] = to_float<T>(x[me.at(rule, n + u * nchunks, P, H, W, status)]);
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                float d = v[u] - K;
                s1 += d;
                s2 = fmaf(d, d, s2);
            }
        }
        for (; n < N; n += nchunks) {
            float d = to_float<T>(x[me.at(rule, n, P, H, W, status)]) - K;
            s1 += d;
            s2 = fmaf(d, d, s2);
        }
    }
    Moments m = from_shifted_sums(cnt, K, s1, s2);
    s_mean[threadIdx.x] = m.mean;
    s_m2[threadIdx.x] = m.m2;
    __syncthreads();
    fold_moments(s_mean, s_m2, cnt, TileChannels(tile, kThreads, Pc, PP), PP,
                 S.partials + (static_cast<size_t>(ck) * tiles + tile) * S.L.max_slots);
}

// ------------------------------------------------------------------------------------ finalize kernels
// One warp per channel; used when the producers did not combine the partials themselves.
__global__ void __launch_bounds__(kThreads)
finalize_stats_kernel(StatsSink S, int C, int HW) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (c >= C) return;
    warp_finish_stats(S, c, HW, threadIdx.x & 31);
}

__global__ void __launch_bounds__(kThreads)
finalize_bwd_kernel(GradSink G, int C, int HW) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * (kThreads / 32) + (threadIdx.x >> 5);
    if (c >= C) return;
    warp_finish_grads(G, c, HW, threadIdx.x & 31);
}

// ------------------------------------------------------------------------------------ normalise + affine
// y = a_c x + b_c with a_c = gamma_c invstd_c and b_c = beta_c - mean_c a_c, over the rows of the chunk.
// With ACT the step that follows a BN layer in a residual network is fused in, so that the pre-activation
// tensor is never written: y = max(0, a x + b + r), r = `res` (may be NULL).
template <typename T, int V, bool ACT>
__device__ __forceinline__ void normalize_rows(const typename T::storage* __restrict__ x,
                                               const typename T::storage* __restrict__ res,
                                               typename T::storage* __restrict__ y, const float* __restrict__ gamma,
                                               const float* __restrict__ beta, const float* __restrict__ mean,
                                               const float* __restrict__ invstd, RowOrder order, int nchunks,
                                               unsigned tiles, int HW, unsigned P) {
    const unsigned tile = blockIdx.x % tiles;
    const int ck = static_cast<int>(blockIdx.x / tiles);
    const unsigned p = (tile * kThreads + threadIdx.x) * V;
    const typename T::storage* xp = x + p;
    const typename T::storage* rp = ACT && res ? res + p : nullptr;
    typename T::storage* yp = y + p;
    // x (and the residual) are inputs of the whole call, so the first rows can be requested before the
    // statistics kernels ahead of this one have finished; only mean / invstd have to wait for them.
    // Rows go in batches of kUnroll with all loads of a batch in flight together; the last batch may be short.
    int i = ck;
    Vec<T, V> v[kUnroll], vr[kUnroll];
    int row[kUnroll];
    if (p < P) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (i + u * nchunks < order.rows) {
                row[u] = order(i + u * nchunks);
                v[u].load(xp + static_cast<size_t>(row[u]) * P);
                if (ACT && rp) vr[u].load(rp + static_cast<size_t>(row[u]) * P);
            }
        }
    }
    grid_dependency_wait();
    grid_dependency_launch();
    if (p >= P) return;
    float a[V], b[V];
    {
        int c[V];
        position_channels<V>(p, HW, c);
#pragma unroll
        for (int j = 0; j < V; ++j) {
            a[j] = gamma[c[j]] * invstd[c[j]];
            b[j] = fmaf(-mean[c[j]], a[j], beta[c[j]]);
        }
    }
    while (true) {
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (i + u * nchunks < order.rows) {
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    float z = fmaf(a[j], v[u].get(j), b[j]);
                    if (ACT) {
                        if (rp) z += vr[u].get(j);
                        z = fmaxf(z, 0.f);
                    }
                    v[u].set(j, z);
                }
                v[u].store(yp + static_cast<size_t>(row[u]) * P);
            }
        }
        i += kUnroll * nchunks;
        if (i >= order.rows) break;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (i + u * nchunks < order.rows) {
                row[u] = order(i + u * nchunks);
                v[u].load(xp + static_cast<size_t>(row[u]) * P);
                if (ACT && rp) vr[u].load(rp + static_cast<size_t>(row[u]) * P);
            }
        }
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
col_normalize_kernel(const typename T::storage* __restrict__ x, typename T::storage* __restrict__ y,
                     const float* __restrict__ gamma, const float* __restrict__ beta, const float* __restrict__ mean,
                     const float* __restrict__ invstd, RowOrder order, int nchunks, unsigned tiles, int HW, unsigned P) {
    normalize_rows<T, V, false>(x, nullptr, y, gamma, beta, mean, invstd, order, nchunks, tiles, HW, P);
}

// ------------------------------------------------------------------------------------ backward, pass 1
// Folds per-THREAD sums into one (sum dy, sum dy (x - mean)) pair per channel the tile meets, for tiles
// whose threads hold V consecutive positions of maps at least V positions large: a thread then meets at
// most two channels, c0 (its first position's) and, if its positions straddle a map boundary, c0 + 1.
// s_first[t] holds thread t's sums over its positions in c0, s_second[t] those in c0 + 1 (zero unless it
// straddles).  The threads of a channel are consecutive, so a slot's total is the sum of s_first over a
// range of threads plus s_second of the one thread just before that range when it straddles into it.
template <int V>
__device__ __forceinline__ void fold_thread_sums(const float2* s_first, const float2* s_second, const TileChannels& tc,
                                                 int HW, float2* out) {
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int slot = warp; slot < tc.nslots; slot += kThreads / 32) {
        unsigned lo, hi;  // positions of the slot's channel inside the tile, relative to its first position
        tc.range(slot, HW, lo, hi);
        const int t_lo = static_cast<int>((lo + V - 1) / V);  // first thread whose first position lies in the channel
        const int t_hi = static_cast<int>((hi + V - 1) / V);
        float sa = 0.f, sb = 0.f;
        for (int t = t_lo + lane; t < t_hi; t += 32) {
            const float2 v = s_first[t];
            sa += v.x;
            sb += v.y;
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            sa += __shfl_down_sync(0xffffffffu, sa, d);
            sb += __shfl_down_sync(0xffffffffu, sb, d);
        }
        if (lane == 0) {
            if (lo % V != 0) {  // the thread before t_lo starts in the previous channel and ends in this one
                const float2 v = s_second[t_lo - 1];
                sa += v.x;
                sb += v.y;
            }
            out[slot] = make_float2(sa, sb);
        }
    }
}

// Streams dy and x once: per channel partial sums of dy and dy (x - mean) and, if WRITE_DX, the
// gradient of every element without the statistics terms, dx = gamma invstd dy (lower branch of Eq. 6).
// PER_CHANNEL selects how a thread keeps its sums when every map holds at least V positions: per channel
// (few registers, four blocks per SM even for bf16; pays extra arithmetic in every warp that holds a
// thread straddling two maps - right for large maps, where such threads are rare) or per position (no
// special case for straddling threads - right for small maps, where most warps hold one).
// With ACT (per-position sums only) the layer is followed by the fused residual add + ReLU: the gradient that
// enters every formula is g = dy where a x + b + r > 0, else 0 (the mask is recomputed from x and r instead
// of being stored), and dr = g is written to `dres` when given.
template <typename T, int V, bool WRITE_DX, bool PER_CHANNEL, bool ACT>
__device__ __forceinline__ void bwd_reduce_rows(const typename T::storage* __restrict__ x,
                                                const typename T::storage* __restrict__ res,
                                                const typename T::storage* __restrict__ dy,
                                                typename T::storage* __restrict__ dx,
                                                typename T::storage* __restrict__ dres,
                                                const float* __restrict__ gamma, const float* __restrict__ beta,
                                                const float* __restrict__ mean, const float* __restrict__ invstd,
                                                RowOrder order, int nchunks, unsigned tiles, int HW, unsigned P,
                                                bool virtual_pass, GradSink G) {
    static_assert(!ACT || (WRITE_DX && !PER_CHANNEL), "the fused activation uses the per-position sums");
    constexpr unsigned TP = kThreads * V;
    // per-position sums (maps smaller than a vector) or, reusing the space, per-thread sums
    __shared__ __align__(16) float s_sums[2 * TP];
    grid_dependency_wait();
    grid_dependency_launch();
    const unsigned tile = blockIdx.x % tiles;
    const int ck = static_cast<int>(blockIdx.x / tiles);
    const unsigned p = (tile * kThreads + threadIdx.x) * V;
    float2* out = (virtual_pass ? G.partials_v : G.partials) +
                  (static_cast<size_t>(ck) * tiles + tile) * (virtual_pass ? G.Lv.max_slots : G.L.max_slots);
    const typename T::storage* xp = x + p;
    const typename T::storage* gp = dy + p;
    typename T::storage* op = WRITE_DX ? dx + p : nullptr;
    if (PER_CHANNEL) {
        // Sums of g and of g (x - pivot) with the pivot the mean of the thread's first channel (one register
        // instead of a mean per position); the deviation from each channel's own mean is put right after the
        // loop: sum g (x - mean) = sum g (x - pivot) - (mean - pivot) sum g.
        // Every thread sums over all its V positions with packed fp32x2 arithmetic (one packed accumulator
        // per sum).  The rare thread whose positions straddle two channels also sums the second channel's
        // share on the side, element by element, inside the same loop - the loads are shared, so a warp that
        // holds such a thread only executes some more arithmetic.
        constexpr int Q = V >= 2 ? V / 2 : 1;
        float2* s_first = reinterpret_cast<float2*>(s_sums);
        float2* s_second = s_first + kThreads;
        float2 first = make_float2(0.f, 0.f), second = make_float2(0.f, 0.f);
        if (p < P) {
            const TwoChannels ch(p, HW, V);
            const bool straddle = ch.jb < V;
            const float mu0 = mean[ch.c0], mu1 = mean[ch.c1];
            const float a0 = WRITE_DX ? gamma[ch.c0] * invstd[ch.c0] : 0.f;
            const float a1 = WRITE_DX ? gamma[ch.c1] * invstd[ch.c1] : 0.f;
            const pair_t minus_pivot = make_pair(-mu0, -mu0);
            const pair_t a2 = make_pair(a0, a0);
            pair_t sum_g = make_pair(0.f, 0.f), sum_gx = make_pair(0.f, 0.f);
            float s1_g = 0.f, s1_gx = 0.f;  // share of channel c1 (positions j >= jb)
            // batches of kUnroll rows, all loads of a batch in flight together; the last batch may be short
            for (int i = ck; i < order.rows; i += kUnroll * nchunks) {
                Vec<T, V> vx[kUnroll], vg[kUnroll];
                int row[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    if (i + u * nchunks < order.rows) {
                        row[u] = order(i + u * nchunks);
                        vx[u].load(xp + static_cast<size_t>(row[u]) * P);
                        vg[u].load(gp + static_cast<size_t>(row[u]) * P);
                    }
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    if (i + u * nchunks < order.rows) {
                        pair_t g2[Q];
#pragma unroll
                        for (int q = 0; q < Q; ++q) {
                            g2[q] = vec_pair<T, V>(vg[u], q);
                            sum_gx = fma2(g2[q], add2(vec_pair<T, V>(vx[u], q), minus_pivot), sum_gx);
                        }
                        if (straddle) {
#pragma unroll
                            for (int q = 0; q < Q; ++q) {
                                float g[2];
                                split_pair(g2[q], g[0], g[1]);
#pragma unroll
                                for (int h = 0; h < 2; ++h) {
                                    const bool in_second = 2 * q + h >= ch.jb;
                                    s1_g += in_second ? g[h] : 0.f;
                                    s1_gx = fmaf(in_second ? g[h] : 0.f, vx[u].get(2 * q + h) - mu0, s1_gx);
                                    if (WRITE_DX) g[h] *= in_second ? a1 : a0;
                                }
                                if (WRITE_DX) set_vec_pair<T, V>(vg[u], q, make_pair(g[0], g[1]));
                            }
                        } else if (WRITE_DX) {
#pragma unroll
                            for (int q = 0; q < Q; ++q) set_vec_pair<T, V>(vg[u], q, mul2(g2[q], a2));
                        }
                        if (WRITE_DX) vg[u].store(op + static_cast<size_t>(row[u]) * P);
#pragma unroll
                        for (int w = Q / 2; w > 0; w >>= 1)
#pragma unroll
                            for (int q = 0; q < w; ++q) g2[q] = add2(g2[q], g2[q + w]);
                        sum_g = add2(sum_g, g2[0]);
                    }
                }
            }
            float lo, hi;
            split_pair(sum_g, lo, hi);
            first.x = lo + hi - s1_g;
            split_pair(sum_gx, lo, hi);
            first.y = lo + hi - s1_gx;
            second = make_float2(s1_g, fmaf(-(mu1 - mu0), s1_g, s1_gx));
        }
        s_first[threadIdx.x] = first;
        s_second[threadIdx.x] = second;
        __syncthreads();
        fold_thread_sums<V>(s_first, s_second, TileChannels(tile, TP, P, HW), HW, out);
    } else {
        // a mean and a pair of sums per position
        float* s_dy = s_sums;
        float* s_dyxc = s_sums + TP;
        float acc_dy[V], acc_dyxc[V];
#pragma unroll
        for (int j = 0; j < V; ++j) acc_dy[j] = acc_dyxc[j] = 0.f;
        if (p < P) {
            float a[V], mu[V], b[V];
            if (HW >= V) {  // at most two channels per thread: two parameter sets, selected per position
                const TwoChannels ch(p, HW, V);
                const float mu0 = mean[ch.c0], mu1 = mean[ch.c1];
                const float a0 = WRITE_DX ? gamma[ch.c0] * invstd[ch.c0] : 0.f;
                const float a1 = WRITE_DX ? gamma[ch.c1] * invstd[ch.c1] : 0.f;
                const float b0 = ACT ? fmaf(-mu0, a0, beta[ch.c0]) : 0.f;
                const float b1 = ACT ? fmaf(-mu1, a1, beta[ch.c1]) : 0.f;
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    mu[j] = ch.pick(j, mu0, mu1);
                    a[j] = ch.pick(j, a0, a1);
                    b[j] = ch.pick(j, b0, b1);
                }
            } else {
                int c[V];
                position_channels<V>(p, HW, c);
#pragma unroll
                for (int j = 0; j < V; ++j) {
                    mu[j] = mean[c[j]];
                    a[j] = WRITE_DX ? gamma[c[j]] * invstd[c[j]] : 0.f;
                    b[j] = ACT ? fmaf(-mu[j], a[j], beta[c[j]]) : 0.f;
                }
            }
            const typename T::storage* rp = ACT && res ? res + p : nullptr;
            typename T::storage* drp = ACT && dres ? dres + p : nullptr;
            for (int i = ck; i < order.rows; i += kUnroll * nchunks) {
                Vec<T, V> vx[kUnroll], vg[kUnroll], vr[kUnroll];
                int row[kUnroll];
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    if (i + u * nchunks < order.rows) {
                        row[u] = order(i + u * nchunks);
                        vx[u].load(xp + static_cast<size_t>(row[u]) * P);
                        vg[u].load(gp + static_cast<size_t>(row[u]) * P);
                        if (ACT && rp) vr[u].load(rp + static_cast<size_t>(row[u]) * P);
                    }
                }
#pragma unroll
                for (int u = 0; u < kUnroll; ++u) {
                    if (i + u * nchunks < order.rows) {
                        float g[V], xv[V];
                        vg[u].unpack(g);
                        vx[u].unpack(xv);
                        if (ACT) {
                            float r[V];
                            if (rp) vr[u].unpack(r);
#pragma unroll
                            for (int j = 0; j < V; ++j)
                                g[j] = fmaf(a[j], xv[j], b[j]) + (rp ? r[j] : 0.f) > 0.f ? g[j] : 0.f;
                            if (drp) {
                                vr[u].pack(g);
                                vr[u].store(drp + static_cast<size_t>(row[u]) * P);
                            }
                        }
#pragma unroll
                        for (int j = 0; j < V; ++j) {
                            acc_dy[j] += g[j];
                            acc_dyxc[j] = fmaf(g[j], xv[j] - mu[j], acc_dyxc[j]);
                            if (WRITE_DX) g[j] *= a[j];
                        }
                        if (WRITE_DX) {
                            vg[u].pack(g);
                            vg[u].store(op + static_cast<size_t>(row[u]) * P);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int j = 0; j < V; ++j) {
            s_dy[threadIdx.x * V + j] = acc_dy[j];
            s_dyxc[threadIdx.x * V + j] = acc_dyxc[j];
        }
        __syncthreads();
        fold_sums(s_dy, s_dyxc, TileChannels(tile, TP, P, HW), HW, out);
    }
}

template <typename T, int V, bool WRITE_DX, bool PER_CHANNEL>
__global__ void __launch_bounds__(kThreads, PER_CHANNEL ? 4 : 3)
col_bwd_reduce_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                      typename T::storage* __restrict__ dx, const float* __restrict__ gamma,
                      const float* __restrict__ mean, const float* __restrict__ invstd, RowOrder order, int nchunks,
                      unsigned tiles, int HW, unsigned P, bool virtual_pass, GradSink G) {
    bwd_reduce_rows<T, V, WRITE_DX, PER_CHANNEL, false>(x, nullptr, dy, dx, nullptr, gamma, nullptr, mean, invstd, order,
                                                        nchunks, tiles, HW, P, virtual_pass, G);
}

// ------------------------------------------------------------------------------------ backward, statistics terms
// Per-channel coefficients of the full gradient of a sampled element (upper branch of Eq. 6):
//   dx = a dy - A - Q (x - mean),  a = gamma invstd,  A = a dbeta / s,  Q = a invstd dgamma / s.
struct FixCoef {
    float a, A, Q, mu;
};

__device__ __forceinline__ FixCoef fix_coef(float gamma, float mean, float invstd, float dgamma, float dbeta,
                                            float inv_s) {
    FixCoef k;
    k.a = gamma * invstd;
    k.A = k.a * dbeta * inv_s;
    k.Q = k.a * invstd * dgamma * inv_s;
    k.mu = mean;
    return k;
}

// masked gradient of one element under the fused residual add + ReLU: dy where the pre-activation is positive
__device__ __forceinline__ float act_gradient(float a, float b, float x, float r, float dy) {
    return fmaf(a, x, b) + r > 0.f ? dy : 0.f;
}

// Rows given by `list` (or begin .. begin+count-1): dx = a dy - A - Q (x - mean); dy == NULL reads as zeros.
// With `fold` the kernel finishes the sums of Eq. 5 itself from the partials in G (see block_finish_grads)
// and dgamma / dbeta are not read.  With ACT the masked gradient takes the place of dy (see bwd_reduce_rows).
template <typename T, int V, bool ACT>
__device__ __forceinline__ void fixup_rows(const typename T::storage* __restrict__ x,
                                           const typename T::storage* __restrict__ res,
                                           const typename T::storage* __restrict__ dy,
                                           typename T::storage* __restrict__ dx, const float* __restrict__ gamma,
                                           const float* __restrict__ beta, const float* __restrict__ mean,
                                           const float* __restrict__ invstd, const float* __restrict__ dgamma,
                                           const float* __restrict__ dbeta, float inv_s, const int* __restrict__ list,
                                           int begin, RowOrder order, int nchunks, unsigned tiles, int HW, unsigned P,
                                           GradSink G, int fold) {
    // rows in flight per thread: the fused activation reads a third tensor, and its pass over a whole tensor
    // (full BN) measured faster with fewer registers and more resident blocks than with deeper batches
    constexpr int U = ACT ? 2 : kUnroll;
    __shared__ float2 s_grad[kFoldSlots];
    grid_dependency_wait();
    grid_dependency_launch();
    const unsigned tile = blockIdx.x % tiles;
    const int ck = static_cast<int>(blockIdx.x / tiles);
    const unsigned p = (tile * kThreads + threadIdx.x) * V;
    const TileChannels tc(tile, kThreads * V, P, HW);
    if (fold) block_finish_grads(G, tc.c_first, tc.nslots, HW, ck == 0, tile, kThreads * V, HW, s_grad);
    if (p >= P) return;
    FixCoef k[V];
    float b[V];
    {
        int c[V];
        position_channels<V>(p, HW, c);
#pragma unroll
        for (int j = 0; j < V; ++j) {
            const float2 g = fold ? s_grad[c[j] - tc.c_first] : make_float2(dgamma[c[j]], dbeta[c[j]]);
            k[j] = fix_coef(gamma[c[j]], mean[c[j]], invstd[c[j]], g.x, g.y, inv_s);
            b[j] = ACT ? fmaf(-k[j].mu, k[j].a, beta[c[j]]) : 0.f;
        }
    }
    const bool with_res = ACT && res;
    int i = ck;
    for (; i + (U - 1) * nchunks < order.rows; i += U * nchunks) {
        Vec<T, V> vx[U], vg[U], vr[U];
        int row[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            int v = order(i + u * nchunks);
            row[u] = list ? list[v] : begin + v;
            vx[u].load(x + static_cast<size_t>(row[u]) * P + p);
            if (dy) vg[u].load(dy + static_cast<size_t>(row[u]) * P + p);
            if (with_res) vr[u].load(res + static_cast<size_t>(row[u]) * P + p);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
#pragma unroll
            for (int j = 0; j < V; ++j) {
                float g = dy ? vg[u].get(j) : 0.f;
                const float xv = vx[u].get(j);
                if (ACT) g = act_gradient(k[j].a, b[j], xv, with_res ? vr[u].get(j) : 0.f, g);
                vg[u].set(j, fmaf(k[j].a, g, -k[j].A) - k[j].Q * (xv - k[j].mu));
            }
            vg[u].store(dx + static_cast<size_t>(row[u]) * P + p);
        }
    }
    for (; i < order.rows; i += nchunks) {
        int v = order(i);
        int n = list ? list[v] : begin + v;
        size_t off = static_cast<size_t>(n) * P + p;
        Vec<T, V> vx, vg, vr;
        vx.load(x + off);
        if (dy) vg.load(dy + off);
        if (with_res) vr.load(res + off);
#pragma unroll
        for (int j = 0; j < V; ++j) {
            float g = dy ? vg.get(j) : 0.f;
            const float xv = vx.get(j);
            if (ACT) g = act_gradient(k[j].a, b[j], xv, with_res ? vr.get(j) : 0.f, g);
            vg.set(j, fmaf(k[j].a, g, -k[j].A) - k[j].Q * (xv - k[j].mu));
        }
        vg.store(dx + off);
    }
}

template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
col_fixup_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                 typename T::storage* __restrict__ dx, const float* __restrict__ gamma, const float* __restrict__ mean,
                 const float* __restrict__ invstd, const float* __restrict__ dgamma, const float* __restrict__ dbeta,
                 float inv_s, const int* __restrict__ list, int begin, RowOrder order, int nchunks, unsigned tiles,
                 int HW, unsigned P, GradSink G, int fold) {
    fixup_rows<T, V, false>(x, nullptr, dy, dx, gamma, nullptr, mean, invstd, dgamma, dbeta, inv_s, list, begin, order,
                            nchunks, tiles, HW, P, G, fold);
}

// The same for the patch elements (compact positions, see PatchThread).
template <typename T, bool ACT>
__device__ __forceinline__ void patch_fixup_rows(const typename T::storage* __restrict__ x,
                                                 const typename T::storage* __restrict__ res,
                                                 const typename T::storage* __restrict__ dy,
                                                 typename T::storage* __restrict__ dx, const float* __restrict__ gamma,
                                                 const float* __restrict__ beta, const float* __restrict__ mean,
                                                 const float* __restrict__ invstd, const float* __restrict__ dgamma,
                                                 const float* __restrict__ dbeta, float inv_s, PatchRule rule, int N,
                                                 int C, int H, int W, int nchunks, unsigned tiles, unsigned* status,
                                                 GradSink G, int fold) {
    __shared__ float2 s_grad[kFoldSlots];
    grid_dependency_wait();
    grid_dependency_launch();
    const unsigned tile = blockIdx.x % tiles;
    const int ck = static_cast<int>(blockIdx.x / tiles);
    const unsigned j = tile * kThreads + threadIdx.x;
    const int PP = rule.ph * rule.pw;
    const TileChannels tc(tile, kThreads, static_cast<unsigned>(C) * PP, PP);  // channels of the tile's compact positions
    if (fold) block_finish_grads(G, tc.c_first, tc.nslots, H * W, ck == 0, tile, kThreads, PP, s_grad);
    if (j >= static_cast<unsigned>(C) * PP) return;
    const PatchThread me(j, rule, H, W);
    const size_t P = static_cast<size_t>(C) * H * W;
    const float2 grads = fold ? s_grad[me.c - tc.c_first] : make_float2(dgamma[me.c], dbeta[me.c]);
    const FixCoef k = fix_coef(gamma[me.c], mean[me.c], invstd[me.c], grads.x, grads.y, inv_s);
    const float b = ACT ? fmaf(-k.mu, k.a, beta[me.c]) : 0.f;
    const bool with_res = ACT && res;
    int n = ck;
    for (; n + (kUnroll - 1) * nchunks < N; n += kUnroll * nchunks) {
        size_t at[kUnroll];
        float g[kUnroll], xv[kUnroll], r[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            at[u] = me.at(rule, n + u * nchunks, P, H, W, status);
            g[u] = to_float<T>(dy[at[u]]);
            xv[u] = to_float<T>(x[at[u]]);
            r[u] = with_res ? to_float<T>(res[at[u]]) : 0.f;
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            if (ACT) g[u] = act_gradient(k.a, b, xv[u], r[u], g[u]);
            dx[at[u]] = from_float<T>(fmaf(k.a, g[u], -k.A) - k.Q * (xv[u] - k.mu));
        }
    }
    for (; n < N; n += nchunks) {
        size_t at = me.at(rule, n, P, H, W, status);
        float g = to_float<T>(dy[at]), xv = to_float<T>(x[at]);
        if (ACT) g = act_gradient(k.a, b, xv, with_res ? to_float<T>(res[at]) : 0.f, g);
        dx[at] = from_float<T>(fmaf(k.a, g, -k.A) - k.Q * (xv - k.mu));
    }
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
patch_fixup_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ dy,
                   typename T::storage* __restrict__ dx, const float* __restrict__ gamma, const float* __restrict__ mean,
                   const float* __restrict__ invstd, const float* __restrict__ dgamma, const float* __restrict__ dbeta,
                   float inv_s, PatchRule rule, int N, int C, int H, int W, int nchunks, unsigned tiles,
                   unsigned* status, GradSink G, int fold) {
    patch_fixup_rows<T, false>(x, nullptr, dy, dx, gamma, nullptr, mean, invstd, dgamma, dbeta, inv_s, rule, N, C, H, W,
                               nchunks, tiles, status, G, fold);
}

// ------------------------------------------------------------------------------------ small sampled sets: one block per channel
// When a channel's sampled set is small (a few thousand elements: small patches, a couple of virtual or
// sampled samples) one block can read all of it, so the statistics need no partials and no finalize
// launch, and in the backward the block that combines the channel's partial sums can apply the
// statistics terms to the channel's sampled elements right away.  SampleSet enumerates the sampled
// elements of a channel as q = 0 .. s-1.
struct SampleSet {
    int patches;       // 1: Feature Sampling patches of the real tensor; 0: whole rows (samples)
    // whole rows: sample indices list[0..rows) or begin .. begin+rows-1; element q = (row q / HW, pixel q % HW)
    const int* list;
    int begin, rows;
    // patches: element q = (sample q / (ph*pw), patch element q % (ph*pw))
    PatchRule patch;
    int N, C, H, W;
    int s;             // elements per channel
    __device__ __forceinline__ size_t at(int c, int q, unsigned* status) const {
        const size_t HW = static_cast<size_t>(H) * W;
        if (patches) {
            const int PP = patch.ph * patch.pw;
            const int n = q / PP, e = q - n * PP;
            const int row = e / patch.pw, col = e - row * patch.pw;
            int oh, ow;
            patch_origin(patch, n, c, H, W, status, oh, ow);
            return (static_cast<size_t>(n) * C + c) * HW + static_cast<size_t>(oh + row) * W + ow + col;
        }
        const int i = q / static_cast<int>(HW), hw = q - i * static_cast<int>(HW);
        const int n = list ? list[i] : begin + i;
        return (static_cast<size_t>(n) * C + c) * HW + hw;
    }
};

// mean and invstd of channel blockIdx.x straight from its sampled elements; if `out` is given, also
// out = gamma (src - mean) invstd + beta on those elements.
constexpr int kDirectUnroll = 12;
// U: loads a thread keeps in flight (sets beyond kUnroll elements per thread take the larger value: fewer
// dependent round trips to memory).
template <typename T, int U = kUnroll>
__global__ void __launch_bounds__(kThreads)
direct_moments_kernel(const typename T::storage* __restrict__ src, SampleSet set, float eps, float* __restrict__ mean,
                      float* __restrict__ invstd, unsigned* status, MovingAverage ma, typename T::storage* __restrict__ out,
                      const float* __restrict__ gamma, const float* __restrict__ beta) {
    __shared__ Moments s_warp[kThreads / 32];
    __shared__ float2 s_affine;
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x;
    float K = 0.f, s1 = 0.f, s2 = 0.f, cnt = 0.f;
    for (int q0 = threadIdx.x; q0 < set.s; q0 += kThreads * U) {
        float v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int q = q0 + u * kThreads;
            if (q < set.s) v[u] = to_float<T>(src[set.at(c, q, status)]);
        }
        if (cnt == 0.f) K = v[0];  // pivot: the thread's first value
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (q0 + u * kThreads < set.s) {
                float d = v[u] - K;
                s1 += d;
                s2 = fmaf(d, d, s2);
                cnt += 1.f;
            }
        }
    }
    Moments m = warp_merge(from_shifted_sums(cnt, K, s1, s2));
    if ((threadIdx.x & 31) == 0) s_warp[threadIdx.x >> 5] = m;
    __syncthreads();
    if (threadIdx.x == 0) {
        Moments acc = s_warp[0];
        for (int w = 1; w < kThreads / 32; ++w) acc = merge(acc, s_warp[w]);
        const float is = 1.0f / sqrtf(acc.m2 / static_cast<float>(set.s) + eps);
        mean[c] = acc.mean;
        invstd[c] = is;
        ma.update(c, acc.mean, acc.m2 / static_cast<float>(set.s));
        if (out) {
            const float a = gamma[c] * is;
            s_affine = make_float2(a, fmaf(-acc.mean, a, beta[c]));
        }
    }
    if (!out) return;
    // the sampled elements themselves are normalised right here (the virtual samples of VDN: the block has
    // just read them, so no separate launch has to)
    __syncthreads();
    const float2 k = s_affine;
    for (int q = threadIdx.x; q < set.s; q += kThreads) {
        const size_t at = set.at(c, q, status);
        out[at] = from_float<T>(fmaf(k.x, to_float<T>(src[at]), k.y));
    }
}

// Backward for a small sampled set: block c combines the partial sums of channel c (as the finalize
// kernel would), publishes dgamma / dbeta, and rewrites the gradient of the channel's sampled elements
// with the statistics terms: dst = a dy - A - Q (src - mean).  dy == NULL reads as zeros; dst == NULL
// skips the rewrite.
template <typename T, int U = kUnroll>
__global__ void __launch_bounds__(kThreads)
direct_finalize_fixup_kernel(const typename T::storage* __restrict__ src, const typename T::storage* __restrict__ dy,
                             typename T::storage* __restrict__ dst, const float* __restrict__ gamma,
                             const float* __restrict__ mean, GradSink G, int HW, SampleSet set, unsigned* status) {
    __shared__ float s_grad[2];
    const int c = blockIdx.x;
    // src and dy are inputs of the whole call (the kernels ahead of this one in the call only write dst and the
    // partial sums), so the first batch of sampled elements is requested before the wait for those kernels.
    // Not when patch locations come from device memory: reading them may raise the status flag, which the
    // call clears just ahead of this kernel.
    const bool early = dst && !(set.patches && set.patch.offsets);
    size_t at[U];
    float g[U], xv[U];
    if (early) {
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const int q = threadIdx.x + u * kThreads;
            if (q < set.s) {
                at[u] = set.at(c, q, status);
                g[u] = dy ? to_float<T>(dy[at[u]]) : 0.f;
                xv[u] = to_float<T>(src[at[u]]);
            }
        }
    }
    // gamma, mean and invstd are inputs of the call as well
    const float scale = gamma[c], mu = mean[c], is = G.invstd[c];
    grid_dependency_wait();
    grid_dependency_launch();
    if (threadIdx.x < 32) {
        const float2 grads = warp_sum_grads(G, c, HW, threadIdx.x);
        if (threadIdx.x == 0) {
            G.dgamma[c] = grads.x;
            G.dbeta[c] = grads.y;
            s_grad[0] = grads.x;
            s_grad[1] = grads.y;
        }
    }
    if (!dst) return;
    __syncthreads();
    const FixCoef k = fix_coef(scale, mu, is, s_grad[0], s_grad[1], 1.0f / static_cast<float>(set.s));
    for (int q0 = threadIdx.x; q0 < set.s; q0 += kThreads * U) {
        if (!(early && q0 == static_cast<int>(threadIdx.x))) {
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int q = q0 + u * kThreads;
                if (q < set.s) {
                    at[u] = set.at(c, q, status);
                    g[u] = dy ? to_float<T>(dy[at[u]]) : 0.f;
                    xv[u] = to_float<T>(src[at[u]]);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u)
            if (q0 + u * kThreads < set.s) dst[at[u]] = from_float<T>(fmaf(k.a, g[u], -k.A) - k.Q * (xv[u] - k.mu));
    }
}

// ------------------------------------------------------------------------------------ per-channel vector kernels
// Eq. 4: statistics mixed from the virtual samples (v) and the sampled real set (s) with weight b on
// the virtual side.  With Var + eps = b (Var_v + eps) + (1-b) (Var_s + eps) the mixed invstd follows
// from the two invstd without ever forming a variance (no cancellation against eps).
__global__ void __launch_bounds__(kThreads)
mix_stats_kernel(const float* __restrict__ mean_s, const float* __restrict__ invstd_s, const float* __restrict__ mean_v,
                 const float* __restrict__ invstd_v, float b, int C, float* __restrict__ mean, float* __restrict__ invstd) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c >= C) return;
    const float is_s = invstd_s[c], is_v = invstd_v[c];
    mean[c] = b * mean_v[c] + (1.0f - b) * mean_s[c];
    invstd[c] = 1.0f / sqrtf(b / (is_v * is_v) + (1.0f - b) / (is_s * is_s));
}

// Eq. 8: moving average of E and Var; the batch variance is recovered from invstd = (Var + eps)^-1/2.
__global__ void __launch_bounds__(kThreads)
moving_average_kernel(const float* __restrict__ mean, const float* __restrict__ invstd, float eps, float alpha, int first,
                      int C, float* __restrict__ mean_ma, float* __restrict__ var_ma) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c >= C) return;
    const float is = invstd[c];
    const float E = mean[c], Var = fmaxf(1.0f / (is * is) - eps, 0.f);
    mean_ma[c] = first ? E : alpha * E + (1.0f - alpha) * mean_ma[c];
    var_ma[c] = first ? Var : alpha * Var + (1.0f - alpha) * var_ma[c];
}

// invstd = (Var + eps)^-1/2 from a recorded variance (validation-time forward).
__global__ void __launch_bounds__(kThreads)
invstd_from_var_kernel(const float* __restrict__ var, float eps, int C, float* __restrict__ invstd) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c < C) invstd[c] = 1.0f / sqrtf(var[c] + eps);
}

// Adds up, in index order, the (dgamma, dbeta) vectors that n row chunks of one layer left behind
// (chunk i at rows[i*2C .. i*2C+C) and rows[i*2C+C .. (i+1)*2C)).
__global__ void __launch_bounds__(kThreads)
sum_chunk_grads_kernel(const float* __restrict__ rows, int n, int C, float* __restrict__ dgamma, float* __restrict__ dbeta) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c >= C) return;
    float g = 0.f, b = 0.f;
    for (int i = 0; i < n; ++i) {
        g += rows[static_cast<size_t>(i) * 2 * C + c];
        b += rows[static_cast<size_t>(i) * 2 * C + C + c];
    }
    dgamma[c] = g;
    dbeta[c] = b;
}

// ------------------------------------------------------------------------------------ statistics shared by several GPUs
// A rank's sampled statistics as (count, mean, M2) rows of C floats, the form in which ranks exchange
// them; rows 1 and 2 arrive holding mean and invstd and row 2 is turned into M2 = count (1/invstd^2 - eps).
__global__ void __launch_bounds__(kThreads)
moments_rows_kernel(float* __restrict__ rows, float count, float eps, int C) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c >= C) return;
    const float is = rows[2 * C + c];
    rows[c] = count;
    rows[2 * C + c] = count * fmaxf(1.0f / (is * is) - eps, 0.f);
}

// Merges the (count, mean, M2) rows of R ranks (rank-major: [R][3][C]) in rank order.
__global__ void __launch_bounds__(kThreads)
merge_rank_moments_kernel(const float* __restrict__ rows, int R, int C, float eps, float* __restrict__ mean,
                          float* __restrict__ invstd, float* __restrict__ count) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c >= C) return;
    Moments acc = {0.f, 0.f, 0.f};
    for (int r = 0; r < R; ++r) {
        const float* q = rows + static_cast<size_t>(r) * 3 * C;
        acc = merge(acc, Moments{q[c], q[C + c], q[2 * C + c]});
    }
    mean[c] = acc.mean;
    invstd[c] = 1.0f / sqrtf(acc.m2 / acc.cnt + eps);
    if (count) count[c] = acc.cnt;  // sampled points per channel over all ranks
}

// The summed backward rows (sum dy, sum dy xhat) of all ranks divided by the merged sampled count: the
// per-point shares that the upper branch of Eq. 6 subtracts.
__global__ void __launch_bounds__(kThreads)
per_point_shares_kernel(const float* __restrict__ sums, const float* __restrict__ count, int C, float* __restrict__ shares) {
    grid_dependency_wait();
    grid_dependency_launch();
    const int c = blockIdx.x * kThreads + threadIdx.x;
    if (c >= C) return;
    const float inv = 1.0f / count[c];
    shares[c] = sums[c] * inv;
    shares[C + c] = sums[C + c] * inv;
}

// ------------------------------------------------------------------------------------ BN + residual add + ReLU
// The step that follows a BN layer in a residual network, fused so that the pre-activation tensor is
// never written: forward y = max(0, a x + b + r); backward g = dy where a x + b + r > 0, else 0, and g
// takes the place of dy everywhere (sums, dx, statistics terms); dr = g.  The mask is recomputed from
// x (and r) instead of being stored.  r / dr may be NULL.  These are the ACT instances of the bodies of
// col_normalize, col_bwd_reduce, col_fixup and patch_fixup.
template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
act_normalize_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ res,
                     typename T::storage* __restrict__ y, const float* __restrict__ gamma,
                     const float* __restrict__ beta, const float* __restrict__ mean, const float* __restrict__ invstd,
                     RowOrder order, int nchunks, unsigned tiles, int HW, unsigned P) {
    normalize_rows<T, V, true>(x, res, y, gamma, beta, mean, invstd, order, nchunks, tiles, HW, P);
}

template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
act_bwd_reduce_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ res,
                      const typename T::storage* __restrict__ dy, typename T::storage* __restrict__ dx,
                      typename T::storage* __restrict__ dres, const float* __restrict__ gamma,
                      const float* __restrict__ beta, const float* __restrict__ mean, const float* __restrict__ invstd,
                      RowOrder order, int nchunks, unsigned tiles, int HW, unsigned P, GradSink G) {
    bwd_reduce_rows<T, V, true, false, true>(x, res, dy, dx, dres, gamma, beta, mean, invstd, order, nchunks, tiles, HW,
                                             P, false, G);
}

template <typename T, int V>
__global__ void __launch_bounds__(kThreads)
act_col_fixup_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ res,
                     const typename T::storage* __restrict__ dy, typename T::storage* __restrict__ dx,
                     const float* __restrict__ gamma, const float* __restrict__ beta, const float* __restrict__ mean,
                     const float* __restrict__ invstd, const float* __restrict__ dgamma, const float* __restrict__ dbeta,
                     float inv_s, const int* __restrict__ list, int begin, RowOrder order, int nchunks, unsigned tiles,
                     int HW, unsigned P, GradSink G, int fold) {
    fixup_rows<T, V, true>(x, res, dy, dx, gamma, beta, mean, invstd, dgamma, dbeta, inv_s, list, begin, order, nchunks,
                           tiles, HW, P, G, fold);
}

template <typename T>
__global__ void __launch_bounds__(kThreads)
act_patch_fixup_kernel(const typename T::storage* __restrict__ x, const typename T::storage* __restrict__ res,
                       const typename T::storage* __restrict__ dy, typename T::storage* __restrict__ dx,
                       const float* __restrict__ gamma, const float* __restrict__ beta, const float* __restrict__ mean,
                       const float* __restrict__ invstd, const float* __restrict__ dgamma,
                       const float* __restrict__ dbeta, float inv_s, PatchRule rule, int N, int C, int H, int W,
                       int nchunks, unsigned tiles, unsigned* status, GradSink G, int fold) {
    patch_fixup_rows<T, true>(x, res, dy, dx, gamma, beta, mean, invstd, dgamma, dbeta, inv_s, rule, N, C, H, W, nchunks,
                              tiles, status, G, fold);
}

// ------------------------------------------------------------------------------------ selection mask (test aid)
__global__ void __launch_bounds__(kThreads)
selection_mask_kernel(uint8_t* __restrict__ mask, int rule, const int* __restrict__ list, int begin, int count,
                      PatchRule patch, int N, int C, int H, int W, unsigned* status) {
    grid_dependency_wait();
    const size_t total = static_cast<size_t>(N) * C * H * W;
    for (size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x; i < total;
         i += static_cast<size_t>(gridDim.x) * kThreads) {
        int w = static_cast<int>(i % W);
        size_t t = i / W;
        int h = static_cast<int>(t % H);
        t /= H;
        int c = static_cast<int>(t % C);
        int n = static_cast<int>(t / C);
        uint8_t in = 0;
        if (rule == 0) {
            in = 1;
        } else if (rule == 1) {
            if (list) {
                for (int j = 0; j < count; ++j) in |= (list[j] == n);
            } else {
                in = n >= begin && n < begin + count;
            }
        } else if (rule == 2) {
            int oh, ow;
            patch_origin(patch, n, c, H, W, status, oh, ow);
            in = h >= oh && h < oh + patch.ph && w >= ow && w < ow + patch.pw;
        }
        mask[i] = in;
    }
}

}  // namespace bns

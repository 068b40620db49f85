// Device code of the V-Major metric and selection (see vmajor_kernels.cu),
// separate from the launch code.
#pragma once
#include "common.cuh"

namespace cocodiff {
namespace vmajor {

constexpr int kMetricThreads = 256;
#ifndef COCODIFF_METRIC_UNROLL
#define COCODIFF_METRIC_UNROLL 4
#endif
#ifndef COCODIFF_METRIC_BLOCKS_PER_SM
#define COCODIFF_METRIC_BLOCKS_PER_SM 4
#endif
constexpr int kMetricUnroll = COCODIFF_METRIC_UNROLL;
constexpr int kMetricBlocksPerSm = COCODIFF_METRIC_BLOCKS_PER_SM;
constexpr int kCountMax = 512;  // groups up to this size are ranked by counting

struct SelectSmem {
    int warp_sums[33];
    int sel_bin, sel_k;
    unsigned long long mstar;
    int t_c;
    unsigned long long stage[kCountMax];  // small groups: the metrics; also reduction slots
};

// Exclusive prefix sum of v over the block; *total receives the block sum.
template <int BLOCK>
__device__ __forceinline__ int block_excl_scan(int v, int *total, int *warp_sums) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int incl = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, incl, off);
        if (lane >= off) incl += t;
    }
    if (lane == 31) warp_sums[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = lane < BLOCK / 32 ? warp_sums[lane] : 0;
        int wi = w;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int t = __shfl_up_sync(0xffffffffu, wi, off);
            if (lane >= off) wi += t;
        }
        if (lane < BLOCK / 32) warp_sums[lane] = wi - w;
        if (lane == 31) warp_sums[32] = wi;
    }
    __syncthreads();
    const int excl = incl - v + warp_sums[warp];
    *total = warp_sums[32];
    __syncthreads();  // warp_sums may be reused by the next scan
    return excl;
}

// Block-wide maximum of a 64-bit value.
template <int BLOCK>
__device__ __forceinline__ unsigned long long block_max_u64(unsigned long long v, unsigned long long *slots) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) {
        const unsigned long long o = __shfl_xor_sync(0xffffffffu, v, off);
        v = o > v ? o : v;
    }
    if (lane == 0) slots[warp] = v;
    __syncthreads();
    unsigned long long r = slots[0];
    for (int w = 1; w < BLOCK / 32; ++w) r = slots[w] > r ? slots[w] : r;
    __syncthreads();
    return r;
}

// Threshold form of the rule: with mstar the metric of the unit of rank
// n_cached-1 in the order (metric, index), unit e is cached iff vals[e] < mstar,
// or vals[e] == mstar and fewer than t_c units equal to mstar precede it.
// Every thread owns a contiguous run of units, so two block scans suffice to
// emit the mask and the ascending list.  vals may live in shared or global memory.
template <int BLOCK>
__device__ void emit_selection(const SelectParams &p, int grp, const unsigned long long *vals, bool none,
                               unsigned long long mstar, int t_c, int *warp_sums) {
    const int tid = threadIdx.x;
    const int g = p.g, base = grp * g, out_base = grp * (g - p.n_cached);
    const int per = (g + BLOCK - 1) / BLOCK;
    const int e_lo = tid * per < g ? tid * per : g;
    const int e_hi = e_lo + per < g ? e_lo + per : g;
    int ties = 0;
    if (!none)
        for (int e = e_lo; e < e_hi; ++e) ties += vals[e] == mstar;
    int scan_total;
    int tie_rank = block_excl_scan<BLOCK>(ties, &scan_total, warp_sums);
    int actives = 0;
    {
        int tr = tie_rank;
        for (int e = e_lo; e < e_hi; ++e) {
            const unsigned long long v = vals[e];
            const bool tie = !none && v == mstar;
            const bool cached = !none && (v < mstar || (tie && tr < t_c));
            tr += tie;
            actives += !cached;
        }
    }
    int pos = block_excl_scan<BLOCK>(actives, &scan_total, warp_sums);
    for (int e = e_lo; e < e_hi; ++e) {
        const unsigned long long v = vals[e];
        const bool tie = !none && v == mstar;
        const bool cached = !none && (v < mstar || (tie && tie_rank < t_c));
        tie_rank += tie;
        if (COCODIFF_IN_BOUNDS(base + e >= 0 && base + e < p.n, p.debug)) p.mask[base + e] = cached ? 0 : 1;
        if (!cached) {
            if (COCODIFF_IN_BOUNDS(out_base + pos >= 0 && out_base + pos < p.n, p.debug)) p.idx[out_base + pos] = base + e;
            ++pos;
        }
    }
    if (grp == 0 && tid == 0) *p.n_active = p.n_groups * (g - p.n_cached);
    __syncthreads();
}

// Small group (g <= kCountMax): every unit is ranked by counting in shared memory.
template <int BLOCK>
__device__ void select_group_small(const SelectParams &p, int grp, SelectSmem &sm) {
    const int tid = threadIdx.x;
    const int g = p.g, n_cached = p.n_cached;
    const unsigned long long *m = p.metric + (long long)grp * g;
    const bool none = n_cached == 0;
    for (int e = tid; e < g; e += BLOCK) sm.stage[e] = m[e];
    __syncthreads();
    if (!none) {
        for (int e = tid; e < g; e += BLOCK) {
            const unsigned long long my = sm.stage[e];
            int less = 0, tie_before = 0;
            for (int j = 0; j < g; ++j) {
                const unsigned long long o = sm.stage[j];
                less += o < my;
                tie_before += (o == my) & (j < e);
            }
            if (less + tie_before == n_cached - 1) { sm.mstar = my; sm.t_c = tie_before + 1; }
        }
        __syncthreads();
    }
    emit_selection<BLOCK>(p, grp, sm.stage, none, none ? 0ull : sm.mstar, none ? 0 : sm.t_c, sm.warp_sums);
}

// Large group: radix select (8 bits per pass, starting at the highest byte in
// use) of the metric of rank n_cached-1.  The metrics are staged in dynamic
// shared memory when they fit (staged != 0); every warp keeps its own histogram
// so that clustered metrics do not serialise the whole block on one counter.
template <int BLOCK>
__device__ void select_group_large(const SelectParams &p, int grp, SelectSmem &sm, unsigned long long *dyn_vals,
                                   int *warp_hist, int staged) {
    const int tid = threadIdx.x, warp = tid >> 5;
    const int g = p.g, n_cached = p.n_cached;
    const unsigned long long *m = p.metric + (long long)grp * g;
    const bool none = n_cached == 0;
    const unsigned long long *vals = m;
    unsigned long long mx = 0;
    for (int e = tid; e < g; e += BLOCK) {
        const unsigned long long v = m[e];
        if (staged) dyn_vals[e] = v;
        mx = v > mx ? v : mx;
    }
    if (staged) vals = dyn_vals;
    mx = block_max_u64<BLOCK>(mx, sm.stage);  // also publishes the staged values
    if (!none) {
        int top = 56;
        while (top > 0 && (mx >> top) == 0ull) top -= 8;
        unsigned long long prefix = 0, pmask = 0;
        int k = n_cached - 1;
        int *my_hist = warp_hist + warp * 256;
        for (int shift = top; shift >= 0; shift -= 8) {
            for (int i = tid; i < (BLOCK / 32) * 256; i += BLOCK) warp_hist[i] = 0;
            __syncthreads();
            for (int e = tid; e < g; e += BLOCK) {
                const unsigned long long v = vals[e];
                if ((v & pmask) == prefix) atomicAdd(&my_hist[(int)((v >> shift) & 255ull)], 1);
            }
            __syncthreads();
            int c = 0;
            if (tid < 256)
                for (int w = 0; w < BLOCK / 32; ++w) c += warp_hist[w * 256 + tid];
            int total;
            const int excl = block_excl_scan<BLOCK>(c, &total, sm.warp_sums);
            if (tid < 256 && c > 0 && excl <= k && k < excl + c) { sm.sel_bin = tid; sm.sel_k = k - excl; }
            __syncthreads();
            prefix |= (unsigned long long)sm.sel_bin << shift;
            pmask |= 0xffull << shift;
            k = sm.sel_k;
            __syncthreads();
        }
        if (tid == 0) { sm.mstar = prefix; sm.t_c = k + 1; }
        __syncthreads();
    }
    emit_selection<BLOCK>(p, grp, vals, none, none ? 0ull : sm.mstar, none ? 0 : sm.t_c, sm.warp_sums);
}

// fix(|a - b|): one fp32 subtraction, scale by 2^16, truncate, saturate to 32
// bits; NaN counts as the saturated value.
__device__ __forceinline__ unsigned fix16(float a, float b) {
    const float d = fabsf(a - b);
    const unsigned r = __float2uint_rz(d * 65536.0f);  // saturating conversion
    return d != d ? 0xffffffffu : r;
}

__device__ __forceinline__ unsigned long long l1_of_vec(const uint4 a, const uint4 b) {
    const unsigned aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    unsigned long long s = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        s += fix16(__uint_as_float(aw[q] << 16), __uint_as_float(bw[q] << 16));
        s += fix16(__uint_as_float(aw[q] & 0xffff0000u), __uint_as_float(bw[q] & 0xffff0000u));
    }
    return s;
}

// Streams this block's share of cur_v / prev_v: warp w of n_warps visits chunks
// w, w + n_warps, ... and adds one 64-bit partial sum per chunk to its unit's
// accumulator.  chunk ids fit 32 bits (checked by the launcher).
__device__ __forceinline__ void metric_stream(const MetricParams &p, const unsigned first_warp, const unsigned n_warps) {
    constexpr int U = kMetricUnroll;
    const int lane = threadIdx.x & 31;
    const unsigned total = (unsigned)p.n_units * (unsigned)p.chunks_per_unit;
    for (unsigned c = first_warp; c < total; c += n_warps) {
        const unsigned u = c / (unsigned)p.chunks_per_unit;
        const unsigned k = c - u * (unsigned)p.chunks_per_unit;
        const long long v0 = (long long)k * p.chunk_vecs;
        const long long v1 = v0 + p.chunk_vecs < p.unit_vecs ? v0 + p.chunk_vecs : p.unit_vecs;
        const uint4 *pc = p.cur + (long long)u * p.unit_vecs;
        const uint4 *pp = p.prev + (long long)u * p.unit_vecs;
        unsigned long long acc = 0;
        for (long long v = v0 + lane; v < v1; v += 32 * U) {
            uint4 a[U], b[U];
#pragma unroll
            for (int i = 0; i < U; ++i)
                if (v + 32 * i < v1) {
                    const bool ok = COCODIFF_IN_BOUNDS((long long)u * p.unit_vecs + v + 32 * i < (long long)p.n_units * p.unit_vecs, p.debug);
                    a[i] = ok ? __ldcs(pc + v + 32 * i) : make_uint4(0, 0, 0, 0);
                    b[i] = ok ? __ldcs(pp + v + 32 * i) : make_uint4(0, 0, 0, 0);
                }
#pragma unroll
            for (int i = 0; i < U; ++i)
                if (v + 32 * i < v1) acc += l1_of_vec(a[i], b[i]);
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0 && acc != 0 && COCODIFF_IN_BOUNDS(u < (unsigned)p.n_units, p.debug)) atomicAdd(p.acc + u, acc);
    }
}

}  // namespace vmajor
}  // namespace cocodiff

// V-Major active-projection selection (Section III-D of the paper, "Active
// projection selection"): an integer L1 distance between the current and the
// cached value vectors per selection unit, then, per group of units, the
// floor(r*g) units with the smallest (distance, index) are marked cached and the
// others active; the active indices are emitted ascending.
//
// metric kernel: streams both tensors once with 128-bit loads; every warp owns
// a contiguous chunk of one unit, reduces with shuffles and adds one 64-bit
// integer per chunk to the unit's accumulator (integer addition: the result
// does not depend on the order).  The block that takes the last ticket copies
// the accumulators out and, for small groups, runs the selection in the same
// launch.  Nothing waits on another block: the ticket is a plain atomic add.
#include "common.cuh"

namespace cocodiff {
namespace {

constexpr int kMetricThreads = 256;
constexpr int kMetricUnroll = 4;
constexpr int kCountMax = 512;  // groups up to this size are ranked by counting

struct SelectSmem {
    int warp_sums[33];
    int hist[256];
    int sel_bin, sel_k;
    unsigned long long mstar;
    int t_c;
    unsigned long long stage[kCountMax];
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

// Selection inside one group, by the whole block.
template <int BLOCK>
__device__ void select_group(const SelectParams &p, int grp, SelectSmem &sm) {
    const int tid = threadIdx.x;
    const int g = p.g, base = grp * g, n_cached = p.n_cached;
    const int out_base = grp * (g - n_cached);
    const unsigned long long *m = p.metric + base;
    const bool none = n_cached == 0;

    // Threshold form of the rule: unit e is cached iff m[e] < mstar, or
    // m[e] == mstar and fewer than t_c equal units precede it.
    if (!none) {
        if (g <= kCountMax) {
            for (int e = tid; e < g; e += BLOCK) sm.stage[e] = m[e];
            __syncthreads();
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
        } else {
            // radix select of the (n_cached-1)-th smallest metric, 8 bits per pass
            unsigned long long prefix = 0, pmask = 0;
            int k = n_cached - 1;
            for (int shift = 56; shift >= 0; shift -= 8) {
                for (int i = tid; i < 256; i += BLOCK) sm.hist[i] = 0;
                __syncthreads();
                for (int e = tid; e < g; e += BLOCK) {
                    const unsigned long long v = m[e];
                    if ((v & pmask) == prefix) atomicAdd(&sm.hist[(int)((v >> shift) & 255ull)], 1);
                }
                __syncthreads();
                const int c = tid < 256 ? sm.hist[tid] : 0;
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
    }
    const unsigned long long mstar = none ? 0ull : sm.mstar;
    const int t_c = none ? 0 : sm.t_c;

    int tie_carry = 0, act_carry = 0;
    for (int c0 = 0; c0 < g; c0 += BLOCK) {
        const int e = c0 + tid;
        const bool valid = e < g;
        const unsigned long long v = valid ? m[e] : 0ull;
        const int tie = (valid && !none && v == mstar) ? 1 : 0;
        int tie_total, act_total;
        const int tie_rank = tie_carry + block_excl_scan<BLOCK>(tie, &tie_total, sm.warp_sums);
        const bool cached = valid && !none && (v < mstar || (tie && tie_rank < t_c));
        const int active = (valid && !cached) ? 1 : 0;
        const int pos = act_carry + block_excl_scan<BLOCK>(active, &act_total, sm.warp_sums);
        if (valid) {
            p.mask[base + e] = (uint8_t)active;
            if (active) p.idx[out_base + pos] = base + e;
        }
        tie_carry += tie_total;
        act_carry += act_total;
    }
    if (grp == 0 && tid == 0) *p.n_active = p.n_groups * (g - n_cached);
    __syncthreads();
}

template <int BLOCK>
__global__ void __launch_bounds__(BLOCK) vmajor_select_kernel(const __grid_constant__ SelectParams p) {
    __shared__ SelectSmem sm;
    select_group<BLOCK>(p, blockIdx.x, sm);
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

__global__ void __launch_bounds__(kMetricThreads, 4)
vmajor_metric_kernel(const __grid_constant__ MetricParams p, const int fuse_select) {
    __shared__ SelectSmem sm;
    __shared__ int is_last;
    constexpr int U = kMetricUnroll;
    const int lane = threadIdx.x & 31;
    // chunk ids fit 32 bits (checked by the launcher): no 64-bit divisions here
    const unsigned warps = gridDim.x * (kMetricThreads / 32);
    const unsigned total = (unsigned)p.n_units * (unsigned)p.chunks_per_unit;
    for (unsigned c = blockIdx.x * (kMetricThreads / 32) + (threadIdx.x >> 5); c < total; c += warps) {
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
                if (v + 32 * i < v1) { a[i] = __ldcs(pc + v + 32 * i); b[i] = __ldcs(pp + v + 32 * i); }
#pragma unroll
            for (int i = 0; i < U; ++i)
                if (v + 32 * i < v1) acc += l1_of_vec(a[i], b[i]);
        }
#pragma unroll
        for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        if (lane == 0 && acc != 0) atomicAdd(p.acc + u, acc);
    }

    // The block that draws the last ticket sees every accumulator complete.
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned t = atomicAdd(p.ticket, 1u);
        is_last = (t == gridDim.x - 1) ? 1 : 0;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    for (int u = threadIdx.x; u < p.n_units; u += kMetricThreads) p.metric[u] = __ldcg(p.acc + u);
    __syncthreads();
    if (fuse_select)
        for (int grp = 0; grp < p.sel.n_groups; ++grp) select_group<kMetricThreads>(p.sel, grp, sm);
}

}  // namespace

cudaError_t launch_select(const SelectParams &p, cudaStream_t stream) {
    if (p.n == 0) {
        return cudaMemsetAsync(p.n_active, 0, sizeof(int32_t), stream);
    }
    if (p.g <= kCountMax)
        vmajor_select_kernel<256><<<p.n_groups, 256, 0, stream>>>(p);
    else
        vmajor_select_kernel<1024><<<p.n_groups, 1024, 0, stream>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_metric_select(const MetricParams &p, cudaStream_t stream) {
    if (p.n_units == 0) return launch_select(p.sel, stream);
    // One resident wave (4 blocks of 256 threads per SM); its warps walk the chunks.
    const long long total = (long long)p.n_units * p.chunks_per_unit;
    if (total > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    long long blocks = (total + (kMetricThreads / 32) - 1) / (kMetricThreads / 32);
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long cap = (long long)sms * 4;
    if (blocks > cap) blocks = cap;
    const int fuse = (p.sel.g <= kCountMax && p.sel.n_groups <= 64) ? 1 : 0;
    vmajor_metric_kernel<<<(unsigned)blocks, kMetricThreads, 0, stream>>>(p, fuse);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || fuse) return e;
    return launch_select(p.sel, stream);
}

}  // namespace cocodiff

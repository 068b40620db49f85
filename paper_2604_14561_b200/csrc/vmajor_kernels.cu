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
        p.mask[base + e] = cached ? 0 : 1;
        if (!cached) p.idx[out_base + pos++] = base + e;
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

__global__ void __launch_bounds__(256) vmajor_select_small_kernel(const __grid_constant__ SelectParams p, const int pdl) {
    __shared__ SelectSmem sm;
    if (pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    select_group_small<256>(p, blockIdx.x, sm);
}

constexpr int kLargeBlock = 1024;
__global__ void __launch_bounds__(kLargeBlock)
vmajor_select_large_kernel(const __grid_constant__ SelectParams p, const int staged, const int pdl) {
    __shared__ SelectSmem sm;
    if (pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    __shared__ int warp_hist[(kLargeBlock / 32) * 256];
    extern __shared__ unsigned long long dyn_vals[];
    select_group_large<kLargeBlock>(p, blockIdx.x, sm, dyn_vals, warp_hist, staged);
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

    // This block has streamed its share: a dependent launch may begin to occupy
    // the SMs (it orders itself behind the whole grid with griddepcontrol.wait).
    if (p.pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

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
        for (int grp = 0; grp < p.sel.n_groups; ++grp) select_group_small<kMetricThreads>(p.sel, grp, sm);
}

}  // namespace

namespace {
template <typename... Args>
cudaError_t launch_maybe_programmatic(void (*kernel)(Args...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                      int pdl, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (pdl & PDL_LAUNCH_ATTR) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}
}  // namespace

cudaError_t launch_select(const SelectParams &p, cudaStream_t stream, int pdl) {
    if (p.n == 0) return cudaMemsetAsync(p.n_active, 0, sizeof(int32_t), stream);
    if (p.g <= kCountMax)
        return launch_maybe_programmatic(vmajor_select_small_kernel, dim3(p.n_groups), dim3(256), 0, stream, pdl, p, pdl);
    // stage the group's metrics in shared memory when they fit beside the histograms
    const size_t want = (size_t)p.g * sizeof(unsigned long long);
    const size_t limit = 160 * 1024;
    const int staged = want <= limit ? 1 : 0;
    const size_t dyn = staged ? want : 0;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64 && !attr_set[dev]) {
        e = cudaFuncSetAttribute(vmajor_select_large_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)limit);
        if (e != cudaSuccess) return e;
        attr_set[dev] = true;
    }
    return launch_maybe_programmatic(vmajor_select_large_kernel, dim3(p.n_groups), dim3(kLargeBlock), dyn, stream, pdl,
                                     p, staged, pdl);
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
    // one small group: its selection rides in the metric kernel's last block; several
    // groups or a large one go to their own launch, one block per group
    const int fuse = (p.sel.g <= kCountMax && p.sel.n_groups <= 2) ? 1 : 0;
    vmajor_metric_kernel<<<(unsigned)blocks, kMetricThreads, 0, stream>>>(p, fuse);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || fuse) return e;
    // the separate selection kernel consumes the metric of the kernel just launched
    return launch_select(p.sel, stream, PDL_LAUNCH_ATTR | PDL_WAIT_AT_START | (p.pdl & PDL_TRIGGER));
}

}  // namespace cocodiff

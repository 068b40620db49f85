// V-Major active-projection selection (Section III-D of the paper, "Active
// projection selection"): an integer L1 distance between the current and the
// cached value vectors per selection unit, then, per group of units, the
// floor(r*g) units with the smallest (distance, index) are marked cached and the
// others active; the active indices are emitted ascending.
//
// metric kernel: streams both tensors once with 128-bit loads.  Large units are
// cut into contiguous pieces, one block per piece, so that the pieces fill one
// resident wave; small units (the per-token rule) take one warp each.  Every
// piece is reduced in registers and shared memory and stored once: no atomics,
// nothing to clear beforehand, and integer addition makes the result
// independent of the order.
//
// selection: up to kCountMax units are ranked by counting - either by every
// block of the kernel that consumes the list (see move_kernels.cu) or by
// vmajor_select_small_kernel; larger groups go to vmajor_select_large_kernel.
#include <mutex>

#include "vmajor.cuh"

namespace cocodiff {
namespace {

using namespace vmajor;

__global__ void __launch_bounds__(256) vmajor_select_small_kernel(const __grid_constant__ SelectParams p, const int pdl) {
    __shared__ SmallSel sm;
    if (pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    select_small<256>(p, (int)blockIdx.x * p.g, p.g, sm, true);  // one group per block
}

__global__ void __launch_bounds__(kLargeBlock)
vmajor_select_large_kernel(const __grid_constant__ SelectParams p, const int mb, const int pdl) {
    __shared__ LargeSel sm;
    extern __shared__ __align__(16) unsigned dyn_words[];
    if (pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // the histogram is cleared while the kernel that produces the metrics still drains
    if (p.n_cached != 0 && p.g <= 65535)
        for (int i = threadIdx.x; i < (int)(large_hist_bytes(mb) / 4); i += kLargeBlock) dyn_words[i] = 0;
    if (pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    select_group_large<kLargeBlock>(p, blockIdx.x, sm, dyn_words, mb);
}

__global__ void __launch_bounds__(kMetricThreads, kMetricBlocksPerSm)
vmajor_metric_kernel(const __grid_constant__ MetricParams p) {
    __shared__ unsigned long long warp_part[kMetricThreads / 32];
    if (p.pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long acc;
    if (p.warp_mode) {
        // one warp per unit, eight consecutive units per block
        const long long u = (long long)blockIdx.x * (kMetricThreads / 32) + warp;
        acc = u < p.n_units ? metric_span(p, u * p.unit_vecs, 0, p.unit_vecs, lane, 32) : 0ull;
    } else {
        // one block per piece of a unit
        const long long u = blockIdx.x / (unsigned)p.parts;
        const long long k = blockIdx.x - u * p.parts;
        const long long v0 = k * p.part_vecs;
        const long long v1 = v0 + p.part_vecs < p.unit_vecs ? v0 + p.part_vecs : p.unit_vecs;
        acc = metric_span(p, u * p.unit_vecs, v0, v1, (int)threadIdx.x, kMetricThreads);
    }
    // This thread has issued all its loads: a dependent launch may begin to occupy
    // the SMs (it orders itself behind the whole grid with griddepcontrol.wait).
    if (p.pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
#pragma unroll
    for (int off = 16; off >= 1; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (p.warp_mode) {
        const long long u = (long long)blockIdx.x * (kMetricThreads / 32) + warp;
        if (lane == 0 && u < p.n_units) p.out[u] = acc;
        return;
    }
    if (lane == 0) warp_part[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned long long s = 0;
#pragma unroll
        for (int w = 0; w < kMetricThreads / 32; ++w) s += warp_part[w];
        p.out[blockIdx.x] = s;
    }
}

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

// Pieces per unit: as many as fill one resident wave of the metric kernel
// (4 blocks on each of 148 SMs), but no piece under 16 KB of each tensor.
// Units of at most 16 KB take one warp each.  The plan depends on the shape
// only, so that it also sizes the workspace.
MetricPlan plan_metric(int n_units, long long unit_vecs) {
    MetricPlan pl;
    pl.parts = 1;
    pl.part_vecs = unit_vecs;
    pl.warp_mode = 0;
    if (n_units <= 0 || unit_vecs <= 0) return pl;
    constexpr long long kWave = 148 * kMetricBlocksPerSm, kMinPiece = 1024, kWarpUnit = 1024;
    if (unit_vecs <= kWarpUnit) {
        pl.warp_mode = 1;
        return pl;
    }
    long long parts = kWave / n_units;
    const long long most = unit_vecs / kMinPiece;
    if (parts > most) parts = most;
    if (parts > 64) parts = 64;
    if (parts < 1) parts = 1;
    pl.parts = (int)parts;
    pl.part_vecs = (unit_vecs + parts - 1) / parts;
    return pl;
}

cudaError_t launch_select(const SelectParams &p, cudaStream_t stream, int pdl) {
    if (p.n == 0) return cudaMemsetAsync(p.n_active, 0, sizeof(int32_t), stream);
    if (p.g <= kCountMax)
        return launch_maybe_programmatic(vmajor_select_small_kernel, dim3(p.n_groups), dim3(256), 0, stream, pdl, p, pdl);
    // the dynamic shared memory needs the opt-in, once per device
    static std::mutex mu;
    static bool attr_set[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaErrorInvalidDevice;
    {
        std::lock_guard<std::mutex> lock(mu);
        if (!attr_set[dev]) {
            e = cudaFuncSetAttribute(vmajor_select_large_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     (int)kLargeDynMax);
            if (e != cudaSuccess) return e;
            attr_set[dev] = true;
        }
    }
    // groups of up to 65535 units keep one 16-bit key per unit behind the histogram; the
    // histogram has 256, 512 or 1024 keys per leading-one position: a narrow one is cleared
    // and scanned faster, a wide one leaves fewer units to tell apart afterwards
    const size_t keys_bytes = p.g <= 65535 ? ((size_t)p.g * 2 + 15) / 16 * 16 : 0;
    int mb = p.g <= 4096 ? 8 : (p.g <= 16384 ? 9 : 10);
    if (large_hist_bytes(mb) + keys_bytes > kLargeDynMax) mb = 9;
    return launch_maybe_programmatic(vmajor_select_large_kernel, dim3(p.n_groups), dim3(kLargeBlock),
                                     large_hist_bytes(mb) + keys_bytes, stream, pdl, p, mb, pdl);
}

cudaError_t launch_metric(const MetricParams &p, cudaStream_t stream) {
    if (p.n_units == 0) return cudaSuccess;
    long long blocks;
    if (p.warp_mode) blocks = ((long long)p.n_units + kMetricThreads / 32 - 1) / (kMetricThreads / 32);
    else blocks = (long long)p.n_units * p.parts;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    return launch_maybe_programmatic(vmajor_metric_kernel, dim3((unsigned)blocks), dim3(kMetricThreads), 0, stream, p.pdl, p);
}

}  // namespace cocodiff

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
#include "vmajor.cuh"

namespace cocodiff {
namespace {

using namespace vmajor;

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

__global__ void __launch_bounds__(kMetricThreads, kMetricBlocksPerSm)
vmajor_metric_kernel(const __grid_constant__ MetricParams p, const int fuse_select) {
    __shared__ SelectSmem sm;
    __shared__ int is_last;
    metric_stream(p, blockIdx.x * (kMetricThreads / 32) + (threadIdx.x >> 5), gridDim.x * (kMetricThreads / 32));

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
    const size_t limit = 188 * 1024;  // with the 37 KB of static shared memory: inside the 227 KB a block may use
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
    const long long cap = (long long)sms * kMetricBlocksPerSm;
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

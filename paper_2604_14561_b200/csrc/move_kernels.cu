// Row mover of the Ulysses prologue: one (token, head) row of D bf16 values is
// read once, optionally RMS-normalised and rotated (Q, K; Section II-B of the
// paper), and written once into its slot of the destination layout (the
// sequence-parallel -> head-parallel exchange of Section II-A, its inverse, the
// compaction of active units and the receiver-side scatter of Section III-D).
//
// A row is D*2 bytes = LPR 16-byte vectors, one per lane of an LPR-lane group,
// so both sides are accessed with full 128-bit vectors and every 32-byte
// sector that is touched is used completely.  A thread keeps its token and
// walks the H heads: the RoPE angles and the norm weight are loaded once per
// token and reused for every head.  No shared memory, no block barrier.
#include "move_rows.cuh"

namespace cocodiff {
namespace {

using namespace rows;

// Runs griddepcontrol.wait when the thread leaves the kernel (any return path).
struct PdlTail {
    int flags;
    __device__ __forceinline__ explicit PdlTail(int f) : flags(f) {}
    __device__ __forceinline__ ~PdlTail() {
        if (flags & PDL_WAIT_AT_END) asm volatile("griddepcontrol.wait;" ::: "memory");
    }
};

// Grid: one block per (job, head range, token tile); THREADS x MINB = threads resident per SM.
template <int LPR, int KIND, int UN, int UP, int THREADS, int MINB, int HINT>
__global__ void __launch_bounds__(THREADS, MINB) move_rows_kernel(const __grid_constant__ MoveParams p) {
    if (p.pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (p.pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    PdlTail tail(p.pdl);  // PDL_WAIT_AT_END: every exit path waits for the predecessor first
    move_block<LPR, KIND, UN, UP, THREADS, HINT>(p, blockIdx.x);
}

// Launch shapes measured on B200 at H = 24, D = 128 (21k tokens): 256 threads,
// 4 blocks per SM (<= 64 registers), evict-first accesses; heads per block and
// loads in flight per thread depend on what the launch contains.
constexpr int kThreads = 256, kMinBlocks = 4, kHint = 0;

template <int LPR, int KIND, int UN, int UP, int THREADS, int MINB, int HINT>
cudaError_t launch_variant(MoveParams p, cudaStream_t stream, int head_split = 1, int order = 1) {
    constexpr int TOK = THREADS / LPR;
    const long long tiles = ((long long)p.n_slots + TOK - 1) / TOK;
    if (head_split < 1) head_split = 1;
    if (head_split > p.H) head_split = p.H;
    p.head_split = head_split;
    p.order = order;
    const long long blocks = tiles * head_split * p.njobs;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (p.pdl & PDL_LAUNCH_ATTR) {
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)blocks);
        cfg.blockDim = dim3(THREADS);
        cfg.stream = stream;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        return cudaLaunchKernelEx(&cfg, move_rows_kernel<LPR, KIND, UN, UP, THREADS, MINB, HINT>, p);
    }
    move_rows_kernel<LPR, KIND, UN, UP, THREADS, MINB, HINT><<<(unsigned)blocks, THREADS, 0, stream>>>(p);
    return cudaGetLastError();
}

// Several blocks per token tile shorten the tail of the grid and let V's plain
// blocks run beside Q/K's arithmetic-heavier ones (head-range-major block order).
template <int LPR>
cudaError_t launch_lpr(const MoveParams &p, cudaStream_t stream) {
    int n_norm = 0;
    for (int i = 0; i < p.njobs; ++i) n_norm += p.job[i].w != nullptr;
    if (n_norm == 0)  // 4 heads per block, 4-8 rows in flight per thread
        return launch_variant<LPR, KIND_PLAIN, 4, 8, kThreads, kMinBlocks, kHint>(p, stream, (p.H + 3) / 4, 1);
    if (n_norm == p.njobs)  // 8 heads per block, 4 rows in flight
        return launch_variant<LPR, KIND_NORM, 4, 8, kThreads, kMinBlocks, kHint>(p, stream, (p.H + 7) / 8, 1);
    // V with Q and/or K in one launch: 12 heads per block, 4 rows in flight on both paths
    return launch_variant<LPR, KIND_MIXED, 4, 4, kThreads, kMinBlocks, kHint>(p, stream, (p.H + 11) / 12, 1);
}

}  // namespace

cudaError_t launch_move(const MoveParams &p, int D, cudaStream_t stream) {
    switch (D) {
        case 32: return launch_lpr<4>(p, stream);
        case 64: return launch_lpr<8>(p, stream);
        case 128: return launch_lpr<16>(p, stream);
        case 256: return launch_lpr<32>(p, stream);
        default: return cudaErrorInvalidValue;
    }
}

// ---------------------------------------------------------------------------
// RoPE angle table, evaluated in double and rounded to float.
namespace {
__global__ void rope_table_kernel(float2 *cs, const int32_t *pos, int S, int D, double theta) {
    const int half = D / 2, n = D / 4;
    const long long total = (long long)S * half;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < total;
         e += (long long)gridDim.x * blockDim.x) {
        const int s = (int)(e / half), pr = (int)(e - (long long)s * half);
        const int axis = pr / n, i = pr - axis * n;
        const double freq = pow(theta, -2.0 * (double)i / (double)half);
        const double phi = (double)pos[2 * s + axis] * freq;
        double sv, cv;
        sincos(phi, &sv, &cv);
        cs[e] = make_float2((float)cv, (float)sv);
    }
}
}  // namespace

cudaError_t launch_rope_table(float *cs, const int32_t *pos, int S, int D, double theta, cudaStream_t stream) {
    const long long total = (long long)S * (D / 2);
    if (total == 0) return cudaSuccess;
    long long blocks = (total + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    rope_table_kernel<<<(unsigned)blocks, 256, 0, stream>>>(reinterpret_cast<float2 *>(cs), pos, S, D, theta);
    return cudaGetLastError();
}

}  // namespace cocodiff

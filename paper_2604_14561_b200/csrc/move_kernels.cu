// Row mover of the Ulysses prologue: one (token, head) row of D bf16 values is
// read once, optionally RMS-normalised and rotated (Q, K; Section II-B of the
// paper), and written once into its slot of the destination layout (the
// sequence-parallel -> head-parallel exchange of Section II-A, its inverse, the
// compaction of active units and the receiver-side scatter of Section III-D).
//
// A row is D*2 bytes = D/8 16-byte vectors, one per lane of an LPR-lane group,
// so both sides are accessed with full 128-bit vectors and every 32-byte
// sector that is touched is used completely.  A thread keeps its token and
// walks the H heads: the RoPE angles and the norm weight are loaded once per
// token and reused for every head.  No shared memory, no block barrier.
//
// selective_move_kernel is the same mover for one selective step (Section
// III-D): when the selection covers at most kCountMax units every block first
// ranks the units itself from the metric kernel's sums (no selection launch and
// no one-block stage between the metric pass and the data movement); an active
// row is then read once and written twice, to the compact send buffer and to its
// slot of the cached head-parallel tensor (or, without a send buffer, to that
// slot alone: direct delivery).
//
// Programmatic dependent launches: a kernel launched with the attribute waits
// (griddepcontrol.wait) before it touches memory and only then lets its own
// successor start, so that nothing it lets start early can overtake the grid it
// waits for; see PdlFlags.
#include <mutex>

#include "move_rows.cuh"
#include "vmajor.cuh"

namespace cocodiff {
namespace {

using namespace rows;

// Launch shapes measured on B200 at H = 24, D = 128 (21k tokens): 256 threads,
// 4 blocks per SM (<= 64 registers), evict-first accesses; heads per block and
// loads in flight per thread depend on what the launch contains.
constexpr int kThreads = 256, kMinBlocks = 4;
// selective mover: rows (heads) requested from the L2 ahead, and the least heads worth a block of its own
constexpr int kSelHeads = 6;

// Grid: one block per (head range, job, token tile); THREADS x MINB = threads resident per SM.
template <int LPR, bool PAD, int KIND, int UN, int UP, bool DUAL = false>
__global__ void __launch_bounds__(kThreads, kMinBlocks) move_rows_kernel(const __grid_constant__ MoveParams p) {
    // wait first: whatever this grid lets start early must not overtake the grid it waits for
    if (p.pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    int n_valid = p.n_slots;
    if (p.map != MAP_FULL) {
        // written by an earlier kernel: a coherent load, ordered after griddepcontrol.wait
        const long long nv = (long long)__ldcg(p.n_active) * p.T;
        n_valid = nv < (long long)p.n_slots ? (int)nv : p.n_slots;
        if (n_valid < 0) n_valid = 0;
    }
    move_block<LPR, PAD, KIND, UN, UP, kThreads, DUAL>(p, blockIdx.x, p.idx, n_valid);
    // A grid that started beside its predecessor without consuming its results still has to
    // complete after it: whoever waits for this grid then also has the predecessor's output.
    if (p.pdl & PDL_WAIT_AT_END) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// The selective mover: 4 blocks of 256 threads per SM.  (One block of 1024 threads ranks the
// units once per SM instead of four times and is 0.4 us faster on 64-token tiles, but slower on
// per-token units and at low cache ratios.)
constexpr int kSelThreads = kThreads, kSelBlocks = kMinBlocks;

template <int LPR, bool PAD>
__global__ void __launch_bounds__(kSelThreads, kSelBlocks)
selective_move_kernel(const __grid_constant__ MoveParams p, const __grid_constant__ SelectParams sel, const int select_here) {
    __shared__ vmajor::SmallSel sm;
    if (p.pdl & PDL_WAIT_AT_START) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.pdl & PDL_TRIGGER) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int32_t *list = p.idx;
    long long nv;
    if (select_here) {
        nv = (long long)vmajor::select_small<kSelThreads>(sel, 0, sel.n, sm, blockIdx.x == 0) * p.T;
        list = sm.idx;
    } else if (p.map == MAP_FULL || p.slots_exact) {
        nv = p.n_slots;  // every slot moves: a plain move, or a grid sized from the rule's own count
    } else {
        nv = (long long)__ldcg(p.n_active) * p.T;
    }
    int n_valid = nv < (long long)p.n_slots ? (int)nv : p.n_slots;
    if (n_valid < 0) n_valid = 0;
    // One resident wave of blocks, so that a block ranks the units once whatever it moves.  The
    // work - for every tensor and every token tile that holds active slots, the H heads - is cut
    // into gridDim.x equal contiguous runs of (tensor, tile, head) rows, heads fastest: a block
    // meets at most two tiles more than its share of heads spans, and no block has more than one
    // head row (of TOK tokens) more than another.  Only the tiles that hold active slots count
    // (the grid's capacity may be larger: the host need not know n_active).
    constexpr unsigned TOK = kSelThreads / LPR;
    const unsigned tiles = ((unsigned)n_valid + TOK - 1) / TOK;
    const unsigned long long total = (unsigned long long)tiles * (unsigned)p.njobs * (unsigned)p.H;
    const unsigned long long per = (total + gridDim.x - 1) / gridDim.x;
    unsigned long long at = per * blockIdx.x;
    const unsigned long long end = at + per < total ? at + per : total;
    while (at < end) {
        const unsigned pair = (unsigned)(at / (unsigned)p.H);        // (tensor, tile), tensor-major
        const int h_lo = (int)(at - (unsigned long long)pair * (unsigned)p.H);
        const int h_hi = (unsigned long long)(p.H - h_lo) < end - at ? p.H : h_lo + (int)(end - at);
        const unsigned job_i = pair / tiles, tile = pair - job_i * tiles;
        move_range<LPR, PAD, KIND_MIXED, 4, 4, kSelThreads, true, kSelHeads>(p, job_i, tile, h_lo, h_hi, list, n_valid);
        at += (unsigned)(h_hi - h_lo);
    }
}

template <typename K, typename... Args>
cudaError_t launch_grid(K kernel, long long blocks, cudaStream_t stream, int pdl, Args... args) {
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (pdl & PDL_LAUNCH_ATTR) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, args...);
}

// multiprocessors of the current device (looked up once per device)
int sm_count() {
    static std::mutex mu;
    static int count[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    std::lock_guard<std::mutex> lock(mu);
    if (count[dev] == 0) {
        int n = 0;
        count[dev] = (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && n > 0) ? n : 148;
    }
    return count[dev];
}

long long grid_blocks(MoveParams &p, int lpr, int heads_per_block) {
    const int tok = kThreads / lpr;
    const long long tiles = ((long long)p.n_slots + tok - 1) / tok;
    int head_split = (p.H + heads_per_block - 1) / heads_per_block;
    if (head_split < 1) head_split = 1;
    if (head_split > p.H) head_split = p.H;
    p.head_split = head_split;
    return tiles * head_split * p.njobs;
}

template <int LPR, bool PAD>
cudaError_t launch_selective_lpr(MoveParams p, const SelectParams *sel, cudaStream_t stream) {
    static const SelectParams none = {};
    // one resident wave, but no more blocks than runs of kSelHeads heads
    constexpr int tok = kSelThreads / LPR;
    const long long tiles = ((long long)p.n_slots + tok - 1) / tok;
    const long long rows = tiles * p.njobs * p.H;
    const long long most = (rows + kSelHeads - 1) / kSelHeads;
    const long long wave = (long long)sm_count() * kSelBlocks;
    p.head_split = 1;
    if (most == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(most < wave ? most : wave));
    cfg.blockDim = dim3(kSelThreads);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = (p.pdl & PDL_LAUNCH_ATTR) ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, selective_move_kernel<LPR, PAD>, p, sel ? *sel : none, sel ? 1 : 0);
}

// Several blocks per token tile shorten the tail of the grid and let V's plain
// blocks run beside Q/K's arithmetic-heavier ones (head-range-major block order).
template <int LPR, bool PAD>
cudaError_t launch_lpr(MoveParams p, cudaStream_t stream) {
    int n_norm = 0, n_dual = 0;
    for (int i = 0; i < p.njobs; ++i) {
        n_norm += p.job[i].w != nullptr;
        n_dual += p.job[i].dst2 != nullptr;
    }
    if (n_dual != 0)  // whole tensors with two destinations: 8 heads per block (92 -> 84 us against the resident wave)
        return n_norm == 0 ? launch_grid(move_rows_kernel<LPR, PAD, KIND_PLAIN, 4, 8, true>, grid_blocks(p, LPR, 8), stream, p.pdl, p)
                           : launch_selective_lpr<LPR, PAD>(p, nullptr, stream);
    // A grid that lets its successor start early does so once its last block has started: when
    // more heads per block make it one resident wave, the successor is launched at once.
    auto heads_per_block = [&](int heads) {
        if (!(p.pdl & PDL_TRIGGER)) return heads;
        const long long tiles = ((long long)p.n_slots + kThreads / LPR - 1) / (kThreads / LPR);
        const long long wave = (long long)sm_count() * kMinBlocks;
        for (int h = 2 * heads; h <= 32 && tiles * ((p.H + heads - 1) / heads) * p.njobs > wave; h *= 2)
            if (tiles * ((p.H + h - 1) / h) * p.njobs <= wave) heads = h;
        return heads;
    };
    if (n_norm == 0)  // 4 heads per block, 4-8 rows in flight per thread
        return launch_grid(move_rows_kernel<LPR, PAD, KIND_PLAIN, 4, 8>, grid_blocks(p, LPR, heads_per_block(4)), stream, p.pdl, p);
    if (n_norm == p.njobs)  // 8 heads per block, 4 rows in flight
        // (the one-wave rule gains 0.4 us on the SD3-class layer here and loses 0.9 us at Qwen 768^2: not applied)
        return launch_grid(move_rows_kernel<LPR, PAD, KIND_NORM, 4, 8>, grid_blocks(p, LPR, 8), stream, p.pdl, p);
    // V with Q and/or K in one launch: 12 heads per block, 4 rows in flight on both paths
    return launch_grid(move_rows_kernel<LPR, PAD, KIND_MIXED, 4, 4>, grid_blocks(p, LPR, 12), stream, p.pdl, p);
}

// D = 8 * lanes; a lane group is padded to the next power of two.
#define COCODIFF_DISPATCH_D(D, CALL)                                   \
    switch (((D) % 8 == 0 && (D) >= 8 && (D) <= 256) ? (D) / 8 : 0) {  \
        case 1: return CALL(1, false);                                 \
        case 2: return CALL(2, false);                                 \
        case 3: return CALL(4, true);                                  \
        case 4: return CALL(4, false);                                 \
        case 5: case 6: case 7: return CALL(8, true);                  \
        case 8: return CALL(8, false);                                 \
        case 9: case 10: case 11: case 12: case 13: case 14: case 15: return CALL(16, true); \
        case 16: return CALL(16, false);                               \
        case 32: return CALL(32, false);                               \
        case 0: return cudaErrorInvalidValue;                          \
        default: return CALL(32, true);                                \
    }

}  // namespace

cudaError_t launch_move(const MoveParams &p, cudaStream_t stream) {
#define CALL_MOVE(LPR, PAD) launch_lpr<LPR, PAD>(p, stream)
    COCODIFF_DISPATCH_D(p.D, CALL_MOVE)
#undef CALL_MOVE
}

cudaError_t launch_selective_move(const MoveParams &p, const SelectParams *sel, cudaStream_t stream) {
#define CALL_SEL(LPR, PAD) launch_selective_lpr<LPR, PAD>(p, sel, stream)
    COCODIFF_DISPATCH_D(p.D, CALL_SEL)
#undef CALL_SEL
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

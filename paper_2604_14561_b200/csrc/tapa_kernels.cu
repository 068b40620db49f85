// Tile-aware parallel all-to-all (TAPA, Section III-B of the paper) on virtual
// ranks: ranks 2g and 2g+1 are the two tiles of GPU g.
//
// Phase 1 (intra-GPU): each tile receives its partner's whole shard, so every
// tile holds all tokens of its GPU.  With the layout p1 = [2][P/2][2*S/P][H][D]
// (p1[t][g] = holdings of tile t of GPU g) each p1[t] is again a [S][H][D]
// tensor: phase 1 is two full copies, done by the row mover (api.cu).
//
// Phase 2 (inter-GPU): one all-to-all per ring t (tile t of every GPU), with
// no traffic between the rings: destination rank r = 2*g2 + t takes its heads
// [r*H/P, (r+1)*H/P) of every token from the copies held by ring t, p1[t].
// This file holds the phase-2 kernel: a row mover whose source tensor depends
// on the ring of the destination head.
#include "common.cuh"

namespace cocodiff {
namespace {

constexpr int kThreads = 256;

// One block: TOK = 256 / LPR tokens, heads [blockIdx.y * hpb, ...) of tensor blockIdx.z.
// A row is D/8 16-byte vectors, one per lane of an LPR-lane group; when D/8 is
// not a power of two the group is padded and its last lanes stay idle.
template <int LPR>
__global__ void __launch_bounds__(kThreads) tapa_phase2_kernel(const __grid_constant__ TapaParams p) {
    const int D = p.D;
    constexpr int TOK = kThreads / LPR;
    const int s = (int)blockIdx.x * TOK + (int)threadIdx.x / LPR;
    if (s >= p.S) return;
    const int lr = (int)threadIdx.x % LPR;
    if (lr >= D / 8) return;
    const uint16_t *src = blockIdx.z == 0 ? p.src[0] : (blockIdx.z == 1 ? p.src[1] : p.src[2]);
    uint16_t *dst = blockIdx.z == 0 ? p.dst[0] : (blockIdx.z == 1 ? p.dst[1] : p.dst[2]);
    const long long E = (long long)p.S * p.H * D;
    const int h_lo = (int)blockIdx.y * p.heads_per_block;
    const int h_hi = h_lo + p.heads_per_block < p.H ? h_lo + p.heads_per_block : p.H;
    for (int h0 = h_lo; h0 < h_hi; h0 += 4) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int h = h0 + u;
            if (h < h_hi) {
                const int ring = (h / p.Hl) & 1;  // destination rank r = h / Hl sits on ring r % 2
                const long long off = ring * E + ((long long)s * p.H + h) * D + 8 * lr;
                v[u] = COCODIFF_IN_BOUNDS(off >= 0 && off + 8 <= 2 * E, p.debug)
                           ? __ldcs(reinterpret_cast<const uint4 *>(src + off)) : make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int h = h0 + u;
            if (h < h_hi) {
                const long long off = ((long long)h * p.S + s) * D + 8 * lr;
                if (COCODIFF_IN_BOUNDS(off >= 0 && off + 8 <= E, p.debug)) __stcs(reinterpret_cast<uint4 *>(dst + off), v[u]);
            }
        }
    }
}

template <int LPR>
cudaError_t launch_lpr(const TapaParams &p, cudaStream_t stream) {
    constexpr int TOK = kThreads / LPR;
    const long long tiles = ((long long)p.S + TOK - 1) / TOK;
    if (tiles == 0 || p.n == 0) return cudaSuccess;
    if (tiles > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    const int split = (p.H + p.heads_per_block - 1) / p.heads_per_block;
    tapa_phase2_kernel<LPR><<<dim3((unsigned)tiles, (unsigned)split, (unsigned)p.n), kThreads, 0, stream>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_tapa_phase2(const TapaParams &p, cudaStream_t stream) {
    if (p.D % 8 != 0 || p.D < 8 || p.D > 256) return cudaErrorInvalidValue;
    const int lanes = p.D / 8;
    if (lanes <= 1) return launch_lpr<1>(p, stream);
    if (lanes <= 2) return launch_lpr<2>(p, stream);
    if (lanes <= 4) return launch_lpr<4>(p, stream);
    if (lanes <= 8) return launch_lpr<8>(p, stream);
    if (lanes <= 16) return launch_lpr<16>(p, stream);
    return launch_lpr<32>(p, stream);
}

}  // namespace cocodiff

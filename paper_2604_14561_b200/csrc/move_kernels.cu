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
#include <cuda_bf16.h>

#include "common.cuh"

namespace cocodiff {
namespace {

constexpr int kThreads = 256;

__device__ __forceinline__ void unpack8(const uint4 v, float (&x)[8]) {
    x[0] = __uint_as_float(v.x << 16);
    x[1] = __uint_as_float(v.x & 0xffff0000u);
    x[2] = __uint_as_float(v.y << 16);
    x[3] = __uint_as_float(v.y & 0xffff0000u);
    x[4] = __uint_as_float(v.z << 16);
    x[5] = __uint_as_float(v.z & 0xffff0000u);
    x[6] = __uint_as_float(v.w << 16);
    x[7] = __uint_as_float(v.w & 0xffff0000u);
}

// two floats -> packed bf16x2, round to nearest even, lo in the low half
__device__ __forceinline__ unsigned pack2(float lo, float hi) {
    const __nv_bfloat162 b = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const unsigned *>(&b);
}

template <int LPR>
__device__ __forceinline__ float group_sum(float v, unsigned mask) {
#pragma unroll
    for (int off = LPR / 2; off >= 1; off >>= 1) v += __shfl_xor_sync(mask, v, off);
    return v;
}

// What a launch may contain: plain moves only, norm + RoPE jobs only, or both
// (the lump order of issue).  The specialised forms need fewer registers.
enum JobKind : int { KIND_PLAIN = 0, KIND_NORM = 1, KIND_MIXED = 2 };

// LPR lanes per row (D = 8 * LPR), UN / UP = heads in flight per thread on the
// norm path / the plain path.
template <int LPR, int KIND, int UN, int UP>
__global__ void __launch_bounds__(kThreads, 4) move_rows_kernel(const __grid_constant__ MoveParams p) {
    constexpr int D = LPR * 8;
    constexpr int TOK = kThreads / LPR;  // token slots per block

    const int tiles = (p.n_slots + TOK - 1) / TOK;
    const int job_i = blockIdx.x / tiles;
    const int tile = blockIdx.x - job_i * tiles;
    const MoveJob job = job_i == 0 ? p.job[0] : (job_i == 1 ? p.job[1] : p.job[2]);

    int n_valid = p.n_slots;
    long long src_head = p.src_head, dst_head = p.dst_head;
    if (p.map != MAP_FULL) {
        const long long nv = (long long)__ldg(p.n_active) * p.T;
        n_valid = nv < (long long)p.n_slots ? (int)nv : p.n_slots;
        if (n_valid < 0) n_valid = 0;
        if (src_head == COMPACT_STRIDE) src_head = (long long)n_valid * D;
        if (dst_head == COMPACT_STRIDE) dst_head = (long long)n_valid * D;
    }

    const int o = tile * TOK + (int)threadIdx.x / LPR;
    const int lr = (int)threadIdx.x % LPR;
    if (o >= n_valid) return;  // whole LPR-lane groups leave together

    long long s = o, d = o;
    if (p.map != MAP_FULL) {
        const int a = o / p.T;
        const long long t = (long long)__ldg(p.idx + a) * p.T + (o - a * p.T);
        if (p.map == MAP_GATHER) s = t; else d = t;
    }

    const uint4 *sp = reinterpret_cast<const uint4 *>(job.src + s * p.src_tok) + lr;
    uint4 *dp = reinterpret_cast<uint4 *>(job.dst + d * p.dst_tok) + lr;
    const long long sh = src_head / 8, dh = dst_head / 8;  // head strides in vectors
    const int H = p.H;

    if (KIND == KIND_PLAIN || (KIND == KIND_MIXED && job.w == nullptr)) {
        int h = 0;
        for (; h + UP <= H; h += UP) {
            uint4 v[UP];
#pragma unroll
            for (int u = 0; u < UP; ++u) { v[u] = __ldcs(sp); sp += sh; }
#pragma unroll
            for (int u = 0; u < UP; ++u) { __stcs(dp, v[u]); dp += dh; }
        }
        for (; h < H; ++h) { __stcs(dp, __ldcs(sp)); sp += sh; dp += dh; }
        return;
    }

    float w[8];
    unpack8(__ldg(reinterpret_cast<const uint4 *>(job.w) + lr), w);
    float c[4] = {1.f, 1.f, 1.f, 1.f}, sn[4] = {0.f, 0.f, 0.f, 0.f};
    if (p.cs != nullptr) {
        // pairs 4*lr .. 4*lr+3 of token s: 8 floats (cos, sin, cos, sin, ...)
        const float4 *t = reinterpret_cast<const float4 *>(p.cs + s * D) + 2 * lr;
        const float4 t0 = __ldg(t), t1 = __ldg(t + 1);
        c[0] = t0.x; sn[0] = t0.y; c[1] = t0.z; sn[1] = t0.w;
        c[2] = t1.x; sn[2] = t1.y; c[3] = t1.z; sn[3] = t1.w;
    }
    const unsigned lane = threadIdx.x & 31u;
    const unsigned gmask = LPR == 32 ? 0xffffffffu : (((1u << LPR) - 1u) << (lane & ~(unsigned)(LPR - 1)));
    const float inv_d = 1.0f / (float)D;
    const float eps = p.eps;

    auto norm_rope_row = [&](const uint4 v) -> uint4 {
        float x[8];
        unpack8(v, x);
        float ss = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) ss = fmaf(x[j], x[j], ss);
        ss = group_sum<LPR>(ss, gmask);
        const float inv = 1.0f / sqrtf(fmaf(ss, inv_d, eps));
        unsigned out[4];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float a = x[2 * q] * inv * w[2 * q];
            const float b = x[2 * q + 1] * inv * w[2 * q + 1];
            out[q] = pack2(a * c[q] - b * sn[q], a * sn[q] + b * c[q]);
        }
        return make_uint4(out[0], out[1], out[2], out[3]);
    };

    int h = 0;
    for (; h + UN <= H; h += UN) {
        uint4 v[UN];
#pragma unroll
        for (int u = 0; u < UN; ++u) { v[u] = __ldcs(sp); sp += sh; }
#pragma unroll
        for (int u = 0; u < UN; ++u) { __stcs(dp, norm_rope_row(v[u])); dp += dh; }
    }
    for (; h < H; ++h) { __stcs(dp, norm_rope_row(__ldcs(sp))); sp += sh; dp += dh; }
}

template <int LPR>
cudaError_t launch_lpr(const MoveParams &p, cudaStream_t stream) {
    constexpr int TOK = kThreads / LPR;
    const long long tiles = ((long long)p.n_slots + TOK - 1) / TOK;
    const long long blocks = tiles * p.njobs;
    if (blocks == 0) return cudaSuccess;
    if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    int n_norm = 0;
    for (int i = 0; i < p.njobs; ++i) n_norm += p.job[i].w != nullptr;
    if (n_norm == 0)
        move_rows_kernel<LPR, KIND_PLAIN, 4, 8><<<(unsigned)blocks, kThreads, 0, stream>>>(p);
    else if (n_norm == p.njobs)
        move_rows_kernel<LPR, KIND_NORM, 4, 8><<<(unsigned)blocks, kThreads, 0, stream>>>(p);
    else
        move_rows_kernel<LPR, KIND_MIXED, 4, 8><<<(unsigned)blocks, kThreads, 0, stream>>>(p);
    return cudaGetLastError();
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

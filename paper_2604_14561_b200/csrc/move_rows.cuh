// Device code of the row mover (see move_kernels.cu for the description of the
// kernels built from it): the per-block work, separate from the launch code.
#pragma once
#include <cuda_bf16.h>

#include "common.cuh"

namespace cocodiff {
namespace rows {

// eight bf16 values of a 16-byte vector, widened exactly
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

// 1/sqrt(x) for x > 0 (x = mean square + eps): one MUFU, relative error < 2^-22
__device__ __forceinline__ float rsqrt_approx(float x) {
    float y;
    asm("rsqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// Sum over the LPR lanes that hold one row; the whole warp takes part.
template <int LPR>
__device__ __forceinline__ float group_sum(float v) {
#pragma unroll
    for (int off = LPR / 2; off >= 1; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
    return v;
}

// What a launch may contain: plain moves only, norm + RoPE jobs only, or both
// (the lump order of issue).  The specialised forms need fewer registers.
enum JobKind : int { KIND_PLAIN = 0, KIND_NORM = 1, KIND_MIXED = 2 };

// Streaming accesses: every row is read once and written once, so both use the
// evict-first policy (cache policies measured the same on B200).
__device__ __forceinline__ uint4 ld_row(const uint4 *p) { return __ldcs(p); }
__device__ __forceinline__ void st_row(uint4 *p, const uint4 v) { __stcs(p, v); }

template <int U>
struct UnrollTag { static constexpr int value = U; };

// Walks heads [h, h_hi) in groups of U (all loads of a group are issued before
// its stores), then halves U for what is left, down to single heads.
template <int U, typename F>
__device__ __forceinline__ void heads_loop(int &h, const int h_hi, F &&body) {
    for (; h + U <= h_hi; h += U) body(UnrollTag<U>{});
    if constexpr (U > 1) heads_loop<U / 2>(h, h_hi, body);
}

// Heads [h_lo, h_hi) of one token tile of one tensor (job).
// A row of D bf16 values is D/8 16-byte vectors, one per lane of an LPR-lane
// group (LPR a power of two).  PAD = false: D = 8 * LPR; PAD = true: D/8 < LPR and
// the lanes beyond the row neither load nor store (they add zero to the row's
// sum of squares).  KIND: what the launch contains; UN / UP = heads in flight per
// thread on the norm path / the plain path.  TOK = THREADS / LPR token slots per
// tile.  DUAL: a job may name a second destination (job.dst2) that is written
// in the same pass - the row's slot in the cached head-parallel tensor beside
// the compact buffer, or the second copy of a shard.  idx_list (shared or global
// memory) and n_valid (active token slots) are resolved by the calling kernel.
// PF: source rows (heads) requested from the L2 ahead of the block's own loads.
template <int LPR, bool PAD, int KIND, int UN, int UP, int THREADS, bool DUAL, int PF = 0>
__device__ __forceinline__ void move_range(const MoveParams &p, const unsigned job_i, const unsigned tile, const int h_lo,
                                           const int h_hi, const int32_t *idx_list, const int n_valid) {
    constexpr int TOK = THREADS / LPR;  // token slots per tile
    const int D = PAD ? p.D : LPR * 8;

    long long src_head = p.src_head, dst_head = p.dst_head;
    if (src_head == COMPACT_STRIDE) src_head = (long long)n_valid * D;
    if (dst_head == COMPACT_STRIDE) dst_head = (long long)n_valid * D;
    const int tile0 = (int)tile * TOK;
    if (tile0 >= n_valid) return;  // block-uniform: nothing in this tile
    const long long sh = src_head / 8, dh = dst_head / 8;  // head strides in vectors
    const int lr = (int)threadIdx.x % LPR;
    const bool lane_on = !PAD || lr < D / 8;
    const MoveJob job = job_i == 0 ? p.job[0] : (job_i == 1 ? p.job[1] : p.job[2]);

    // A slot past the end keeps its lanes in step with the warp (the row
    // reduction uses full-warp shuffles): it re-reads the tile's first slot
    // and stores nothing.
    const int o_raw = tile0 + (int)threadIdx.x / LPR;
    const bool valid = o_raw < n_valid;
    const int o = valid ? o_raw : tile0;

    long long s = o, d = o, d2 = o;
    if (p.map != MAP_FULL) {
        const int a = o / p.T;
        (void)COCODIFF_IN_BOUNDS(a >= 0 && a < p.n_units, p.debug);
        int unit = idx_list[a];  // a list that was never written must not send accesses out of bounds
        unit = unit < 0 ? 0 : (unit >= p.n_units ? p.n_units - 1 : unit);
        const long long tk = (long long)unit * p.T + (o - a * p.T);
        if (p.map != MAP_SCATTER) s = tk;
        if (p.map != MAP_GATHER) d = tk;
        d2 = tk;
    }
    // bounds-checked build only: is the 16-byte vector at ptr inside its buffer?
    auto src_ok = [&](const uint4 *ptr) {
        return COCODIFF_IN_BOUNDS(reinterpret_cast<const uint16_t *>(ptr) >= job.src &&
                                  reinterpret_cast<const uint16_t *>(ptr) - job.src + 8 <= p.src_extent, p.debug);
    };
    auto dst_ok = [&](const uint4 *ptr) {
        return COCODIFF_IN_BOUNDS(reinterpret_cast<const uint16_t *>(ptr) >= job.dst &&
                                  reinterpret_cast<const uint16_t *>(ptr) - job.dst + 8 <= p.dst_extent, p.debug);
    };
    auto dst2_ok = [&](const uint4 *ptr) {
        return COCODIFF_IN_BOUNDS(reinterpret_cast<const uint16_t *>(ptr) >= job.dst2 &&
                                  reinterpret_cast<const uint16_t *>(ptr) - job.dst2 + 8 <= p.dst2_extent, p.debug);
    };
    (void)src_ok;
    (void)dst_ok;
    (void)dst2_ok;
    const uint4 *sp = reinterpret_cast<const uint4 *>(job.src + s * p.src_tok) + lr + h_lo * sh;
    uint4 *dp = reinterpret_cast<uint4 *>(job.dst + d * p.dst_tok) + lr + h_lo * dh;
    // second destination, with strides of its own
    const bool dual = DUAL && job.dst2 != nullptr;
    const long long dh2 = DUAL ? p.dst2_head / 8 : 0;
    uint4 *dp2 = DUAL ? reinterpret_cast<uint4 *>(job.dst2 + (dual ? d2 * p.dst2_tok : 0)) + lr + h_lo * dh2 : nullptr;

    // A block that walks a few runs of scattered units meets the memory latency anew at every
    // run (the list, then the per-token constants, then the rows): the rows of the first PF
    // heads are asked of the L2 before the constants are loaded.  (Whole-tensor moves and grids
    // of one range per block hide that latency behind their other work, and measured slower
    // with the extra requests.)
    if (PF > 0 && p.map != MAP_FULL && lane_on) {
        const int np = h_hi - h_lo < PF ? h_hi - h_lo : PF;
        for (int u = 0; u < np; ++u) asm volatile("prefetch.global.L2 [%0];" ::"l"(sp + u * sh));
    }
    if (KIND == KIND_PLAIN || (KIND == KIND_MIXED && job.w == nullptr)) {
        if (!valid || !lane_on) return;
        int h = h_lo;
        heads_loop<UP>(h, h_hi, [&](auto u_tag) {
            constexpr int U = decltype(u_tag)::value;
            uint4 v[U];
#pragma unroll
            for (int u = 0; u < U; ++u) { v[u] = src_ok(sp) ? ld_row(sp) : make_uint4(0, 0, 0, 0); sp += sh; }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (dst_ok(dp)) st_row(dp, v[u]);
                dp += dh;
                if (DUAL) {
                    if (dual && dst2_ok(dp2)) st_row(dp2, v[u]);
                    dp2 += dh2;
                }
            }
        });
        return;
    }

    // Per-token constants, reused for all heads: the norm weight folded into the
    // rotation.  With pair q = elements (2q, 2q+1) = (a_q, b_q):
    //   out[2q] = inv * (a_q*ka_q + b_q*kb_q),  out[2q+1] = inv * (a_q*kc_q + b_q*kd_q).
    // Pairs (0,1) and (2,3) are processed together with sm_100's packed fp32x2
    // arithmetic (two independent IEEE fp32 operations per instruction).
    float2 ka01, kb01, kc01, kd01, ka23, kb23, kc23, kd23;
    {
        float w[8];
        unpack8(lane_on ? __ldg(reinterpret_cast<const uint4 *>(job.w) + lr) : make_uint4(0, 0, 0, 0), w);
        float c[4] = {1.f, 1.f, 1.f, 1.f}, sn[4] = {0.f, 0.f, 0.f, 0.f};
        if (p.cs != nullptr && lane_on) {
            // pairs 4*lr .. 4*lr+3 of token s: 8 floats (cos, sin, cos, sin, ...)
            const float4 *tb = reinterpret_cast<const float4 *>(p.cs + s * D) + 2 * lr;
            const bool cs_ok = COCODIFF_IN_BOUNDS(s >= 0 && s * D + 8 * lr + 8 <= p.cs_extent, p.debug);
            const float4 t0 = cs_ok ? __ldg(tb) : make_float4(1.f, 0.f, 1.f, 0.f);
            const float4 t1 = cs_ok ? __ldg(tb + 1) : make_float4(1.f, 0.f, 1.f, 0.f);
            c[0] = t0.x; sn[0] = t0.y; c[1] = t0.z; sn[1] = t0.w;
            c[2] = t1.x; sn[2] = t1.y; c[3] = t1.z; sn[3] = t1.w;
        }
        ka01 = make_float2(w[0] * c[0], w[2] * c[1]);
        kb01 = make_float2(-(w[1] * sn[0]), -(w[3] * sn[1]));
        kc01 = make_float2(w[0] * sn[0], w[2] * sn[1]);
        kd01 = make_float2(w[1] * c[0], w[3] * c[1]);
        ka23 = make_float2(w[4] * c[2], w[6] * c[3]);
        kb23 = make_float2(-(w[5] * sn[2]), -(w[7] * sn[3]));
        kc23 = make_float2(w[4] * sn[2], w[6] * sn[3]);
        kd23 = make_float2(w[5] * c[2], w[7] * c[3]);
    }
    const float inv_d = 1.0f / (float)D;
    const float eps = p.eps;

    auto norm_rope_row = [&](const uint4 v) -> uint4 {
        // a_q = low bf16 of word q, b_q = high bf16 of word q, widened exactly
        const float2 a01 = make_float2(__uint_as_float(v.x << 16), __uint_as_float(v.y << 16));
        const float2 b01 = make_float2(__uint_as_float(v.x & 0xffff0000u), __uint_as_float(v.y & 0xffff0000u));
        const float2 a23 = make_float2(__uint_as_float(v.z << 16), __uint_as_float(v.w << 16));
        const float2 b23 = make_float2(__uint_as_float(v.z & 0xffff0000u), __uint_as_float(v.w & 0xffff0000u));
        float2 acc = __fmul2_rn(a01, a01);
        acc = __ffma2_rn(b01, b01, acc);
        acc = __ffma2_rn(a23, a23, acc);
        acc = __ffma2_rn(b23, b23, acc);
        const float ss = group_sum<LPR>(acc.x + acc.y);
        const float inv = rsqrt_approx(fmaf(ss, inv_d, eps));
        const float2 inv2 = make_float2(inv, inv);
        const float2 lo01 = __fmul2_rn(__ffma2_rn(a01, ka01, __fmul2_rn(b01, kb01)), inv2);
        const float2 hi01 = __fmul2_rn(__ffma2_rn(a01, kc01, __fmul2_rn(b01, kd01)), inv2);
        const float2 lo23 = __fmul2_rn(__ffma2_rn(a23, ka23, __fmul2_rn(b23, kb23)), inv2);
        const float2 hi23 = __fmul2_rn(__ffma2_rn(a23, kc23, __fmul2_rn(b23, kd23)), inv2);
        return make_uint4(pack2(lo01.x, hi01.x), pack2(lo01.y, hi01.y), pack2(lo23.x, hi23.x), pack2(lo23.y, hi23.y));
    };

    int h = h_lo;
    heads_loop<UN>(h, h_hi, [&](auto u_tag) {
        constexpr int U = decltype(u_tag)::value;
        uint4 v[U];
#pragma unroll
        for (int u = 0; u < U; ++u) { v[u] = (lane_on && src_ok(sp)) ? ld_row(sp) : make_uint4(0, 0, 0, 0); sp += sh; }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint4 y = norm_rope_row(v[u]);
            if (valid && lane_on && dst_ok(dp)) st_row(dp, y);
            dp += dh;
            if (DUAL) {
                if (dual && valid && lane_on && dst2_ok(dp2)) st_row(dp2, y);
                dp2 += dh2;
            }
        }
    });
}

// One block's share of a grid of one block per (head range, job, token tile):
// block id b, head-range-major, so that the V, Q and K tiles of one head range are
// neighbours in the grid and V's plain blocks run beside the arithmetic-heavier
// Q/K blocks.
template <int LPR, bool PAD, int KIND, int UN, int UP, int THREADS, bool DUAL>
__device__ __forceinline__ void move_block(const MoveParams &p, const unsigned b, const int32_t *idx_list,
                                           const int n_valid) {
    constexpr int TOK = THREADS / LPR;
    const unsigned tiles = (unsigned)(p.n_slots + TOK - 1) / TOK;
    const unsigned hsplit = (unsigned)p.head_split, njobs = (unsigned)p.njobs;
    const unsigned y = b / (tiles * njobs);
    const unsigned rem = b - y * tiles * njobs;
    const unsigned job_i = rem / tiles;
    const unsigned tile = rem - job_i * tiles;
    const int hs = (p.H + (int)hsplit - 1) / (int)hsplit;
    const int h_lo = (int)y * hs;
    const int h_hi = h_lo + hs < p.H ? h_lo + hs : p.H;
    move_range<LPR, PAD, KIND, UN, UP, THREADS, DUAL>(p, job_i, tile, h_lo, h_hi, idx_list, n_valid);
}

}  // namespace rows
}  // namespace cocodiff

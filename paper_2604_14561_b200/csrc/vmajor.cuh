// Device code of the V-Major metric and selection (see vmajor_kernels.cu),
// separate from the launch code.
#pragma once
#include "common.cuh"

namespace cocodiff {
namespace vmajor {

constexpr int kMetricThreads = 256;
constexpr int kMetricUnroll = 4;       // 16-byte loads of each tensor in flight per thread
constexpr int kMetricBlocksPerSm = 4;

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

// The metric of unit e: given directly, or the sum of the pieces the metric
// kernel stored.  Written by the preceding kernel of the stream: coherent loads.
__device__ __forceinline__ unsigned long long unit_metric(const SelectParams &p, int e) {
    if (p.parts == 0) return COCODIFF_IN_BOUNDS(e >= 0 && e < p.n, p.debug) ? __ldcg(p.metric + e) : 0ull;
    unsigned long long v = 0;
    for (int k = 0; k < p.parts; ++k)
        if (COCODIFF_IN_BOUNDS(e >= 0 && e < p.n, p.debug)) v += __ldcg(p.partial + (long long)e * p.parts + k);
    return v;
}

// ---------------------------------------------------------------------------
// Up to kCountMax units, whole groups: every unit is ranked inside its group by
// counting (metric, index) pairs in shared memory; the units of rank >= n_cached
// are active.  Leaves the ascending active list in sm.idx and returns its
// length; with publish the block also writes metric_out, mask, idx and n_active.
constexpr int kStageMax = 768;   // piece sums staged at once (units * pieces of the selections that run in a consumer)
struct alignas(16) SmallSel {
    unsigned long long m[kCountMax];
    unsigned long long stage[kStageMax];
    int idx[kCountMax];
    unsigned char active[kCountMax];
    unsigned words[kCountMax / 32];   // the active flags, one bit per unit
    int wide;                         // some metric does not leave room for the index beside it
};

template <int BLOCK>
__device__ int select_small(const SelectParams &p, const int base, const int cnt, SmallSel &sm, const bool publish) {
    const int tid = threadIdx.x, lane = tid & 31;
    if (tid == 0) sm.wide = 0;
    const int n_pieces = cnt * p.parts;
    if (p.parts >= 2 && n_pieces <= kStageMax) {
        // the piece sums: coalesced, and all loads of a thread in flight together
        const unsigned long long *src = p.partial + (long long)base * p.parts;
        unsigned long long v[(kStageMax + BLOCK - 1) / BLOCK];
#pragma unroll
        for (int u = 0; u < (kStageMax + BLOCK - 1) / BLOCK; ++u)
            v[u] = (tid + u * BLOCK < n_pieces && COCODIFF_IN_BOUNDS((long long)base * p.parts + tid + u * BLOCK < (long long)p.n * p.parts, p.debug))
                       ? __ldcg(src + tid + u * BLOCK) : 0ull;
#pragma unroll
        for (int u = 0; u < (kStageMax + BLOCK - 1) / BLOCK; ++u)
            if (tid + u * BLOCK < n_pieces) sm.stage[tid + u * BLOCK] = v[u];
        __syncthreads();
        for (int e = tid; e < cnt; e += BLOCK) {
            unsigned long long sum = 0;
            for (int k = 0; k < p.parts; ++k) sum += sm.stage[e * p.parts + k];
            sm.m[e] = sum;
        }
    } else {
        for (int e = tid; e < cnt; e += BLOCK) sm.m[e] = unit_metric(p, base + e);
    }
    __syncthreads();
    // Rank by counting.  While every metric is below 2^55 the pair (metric, unit) is one 64-bit
    // key and a rank costs one comparison per other unit; else the two fields are compared.
    for (int e = tid; e < cnt; e += BLOCK)
        if (sm.m[e] >> 55) sm.wide = 1;
    __syncthreads();
    static_assert(BLOCK >= kCountMax, "one thread per unit");
    const int e = tid;
    if (!sm.wide) {
        if (e < cnt) sm.stage[e] = (sm.m[e] << 9) | (unsigned long long)e;  // cnt <= 256 < 2^9
        __syncthreads();
        if (e < cnt) {
            const int g0 = (e / p.g) * p.g, g1 = g0 + p.g;  // base is a multiple of g
            const unsigned long long my = sm.stage[e];
            int rank = 0;
            // every warp reads every key of its units' groups, so the loop is bound by the
            // shared-memory pipe: two keys per load
            int j = g0;
            if ((j & 1) && j < g1) rank += sm.stage[j++] < my;
#pragma unroll 4
            for (; j + 2 <= g1; j += 2) {
                const ulonglong2 kk = *reinterpret_cast<const ulonglong2 *>(&sm.stage[j]);
                rank += (kk.x < my) + (kk.y < my);
            }
            if (j < g1) rank += sm.stage[j] < my;
            sm.active[e] = rank >= p.n_cached ? 1 : 0;
        }
    } else if (e < cnt) {
        const int g0 = (e / p.g) * p.g;
        const unsigned long long my = sm.m[e];
        int rank = 0;
        for (int j = g0; j < g0 + p.g; ++j) {
            const unsigned long long o = sm.m[j];
            rank += (o < my) | ((o == my) & (j < e));
        }
        sm.active[e] = rank >= p.n_cached ? 1 : 0;
    }
    __syncthreads();
    const int cnt_pad = (cnt + 31) / 32 * 32;
    for (int e = tid; e < cnt_pad; e += BLOCK) {
        const unsigned w = __ballot_sync(0xffffffffu, e < cnt && sm.active[e]);
        if (lane == 0) sm.words[e >> 5] = w;
    }
    __syncthreads();
    // position of an active unit in the ascending list: the set bits before it
    int total = 0;
    for (int w = 0; w < cnt_pad / 32; ++w) total += __popc(sm.words[w]);
    for (int e = tid; e < cnt; e += BLOCK)
        if (sm.active[e]) {
            int pos = __popc(sm.words[e >> 5] & ((1u << (e & 31)) - 1u));
            for (int w = 0; w < (e >> 5); ++w) pos += __popc(sm.words[w]);
            sm.idx[pos] = base + e;
        }
    __syncthreads();
    if (publish) {
        const int out_base = (base / p.g) * (p.g - p.n_cached);
        for (int e = tid; e < cnt; e += BLOCK)
            if (COCODIFF_IN_BOUNDS(base + e >= 0 && base + e < p.n, p.debug)) {
                p.mask[base + e] = sm.active[e];
                if (p.parts != 0) p.metric_out[base + e] = sm.m[e];
            }
        for (int a = tid; a < total; a += BLOCK)
            if (COCODIFF_IN_BOUNDS(out_base + a >= 0 && out_base + a < p.n, p.debug)) p.idx[out_base + a] = sm.idx[a];
        if (base == 0 && tid == 0) *p.n_active = p.n_groups * (p.g - p.n_cached);
    }
    return total;
}

// ---------------------------------------------------------------------------
// Large group: one block finds the metric of rank n_cached-1 (mstar) and how
// many of the units equal to it are cached (t_c), then emits mask and list.
//
// Groups of at most 65535 units: one pass over the metrics computes a monotone
// key of each 64-bit metric - position of its leading one (6 bits) and the mb
// bits below it (mb = 10, or 9 when that does not fit) -, keeps the keys in
// shared memory as 16-bit values and counts them in a histogram of 16-bit
// counters.  A scan of the histogram gives the key that contains the wanted
// rank; every later pass reads the 2-byte keys and fetches the 8-byte metric
// again only for the few units of that key.  The rank among those units is
// resolved by counting when they are few, else by 8-bit radix passes over the
// bits the key does not cover.  Larger groups skip the keys and run the radix
// passes over all bits in use, reading the metrics from global memory.
constexpr int kLargeBlock = 1024;
constexpr int kCandMax = 256;

struct LargeSel {
    int warp_sums[33];
    int sel_bin, sel_k, sel_owner;
    unsigned long long mstar;
    int t_c;
    int n_cand;
    unsigned long long slots[kLargeBlock / 32];
    unsigned long long cand_val[kCandMax];
    int cand_idx[kCandMax];
    unsigned less_mask[2048], tie_mask[2048];  // one bit per unit, groups of at most 65536 units
    int chunk_pos[2048];                       // active units before each 32-unit chunk
};
// Dynamic shared memory: [histogram of (64 << mb) 16-bit counters, at least 32 KB - it is
// reused as 32 per-warp 256-bin histograms by the radix passes][one 16-bit key per unit].
constexpr size_t kLargeDynMax = 196 * 1024;   // beside the static part: inside the 227 KB a block may use
__host__ __device__ constexpr size_t large_hist_bytes(int mb) { return ((size_t)64 << mb) * 2; }

__device__ __forceinline__ unsigned key_of(unsigned long long v, int mb) {
    if (v < 2) return 0;  // 0 and 1 share the first key
    const int e = 63 - __clzll((long long)v);
    const unsigned long long frac = (v << (63 - e)) << 1;  // bits below the leading one, left-aligned
    return ((unsigned)e << mb) | (unsigned)(frac >> (64 - mb));
}
// smallest metric with that key
__device__ __forceinline__ unsigned long long key_base(unsigned key, int mb) {
    if (key == 0) return 0ull;
    const int e = (int)(key >> mb);
    const unsigned long long top = (1ull << mb) | (key & ((1u << mb) - 1u));  // leading one and mb bits
    return e >= mb ? top << (e - mb) : top >> (mb - e);
}
// number of low bits of the metric that the key leaves open
__device__ __forceinline__ int key_low_bits(unsigned key, int mb) {
    if (key == 0) return 1;
    const int e = (int)(key >> mb);
    return e > mb ? e - mb : 0;
}

// 8-bit radix passes from `shift_top` down to 0 over the units whose key is
// want_key (keys == nullptr: all units); k = wanted rank among them.  Leaves the
// selected low bits in *prefix_out and the rank among equals in *k_out.
template <int BLOCK>
__device__ void radix_passes(const unsigned long long *vals, const unsigned short *keys, int g, unsigned want_key,
                             int shift_top, int k, LargeSel &sm, int *warp_hist, unsigned long long *prefix_out,
                             int *k_out) {
    const int tid = threadIdx.x, warp = tid >> 5;
    unsigned long long prefix = 0, pmask = 0;
    int *my_hist = warp_hist + warp * 256;
    for (int shift = shift_top; shift >= 0; shift -= 8) {
        for (int i = tid; i < (BLOCK / 32) * 256; i += BLOCK) warp_hist[i] = 0;
        __syncthreads();
        for (int e = tid; e < g; e += BLOCK) {
            if (keys != nullptr && keys[e] != want_key) continue;
            const unsigned long long v = __ldcg(vals + e);
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
    *prefix_out = prefix;
    *k_out = k;
}

// Threshold form of the rule: unit e is cached iff vals[e] < mstar, or
// vals[e] == mstar and fewer than t_c units equal to mstar precede it.  The
// metrics are compared once: the "less" and "tie" bits of every 32-unit chunk
// are kept as two words in shared memory.  Then one thread per chunk turns them
// into the chunk's active bits (two block scans over the chunks give the number
// of ties and of active units before each chunk), and a last pass over the units
// writes mask and list.  No pass carries a running count from one iteration to
// the next.  For groups of at most 65536 units.
template <int BLOCK>
__device__ void emit_selection_masks(const SelectParams &p, int grp, const unsigned long long *vals,
                                     const unsigned short *keys, unsigned bin, bool none, unsigned long long mstar,
                                     int t_c, LargeSel &sm) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int WARPS = BLOCK / 32;
    const int g = p.g, base = grp * g, out_base = grp * (g - p.n_cached);
    const int n_chunks = (g + 31) / 32;
    for (int c = warp; c < n_chunks; c += WARPS) {
        const int e = 32 * c + lane;
        bool less = false, tie = false;
        if (!none && e < g) {
            const unsigned key = keys[e];  // a key below / above the selected one decides without the metric
            less = key < bin;
            if (key == bin) {
                const unsigned long long v = __ldcg(vals + e);
                less = v < mstar;
                tie = v == mstar;
            }
        }
        const unsigned lm = __ballot_sync(0xffffffffu, less);
        const unsigned tm = __ballot_sync(0xffffffffu, tie);
        if (lane == 0) { sm.less_mask[c] = lm; sm.tie_mask[c] = tm; }
    }
    __syncthreads();
    // thread t owns chunks 2t and 2t+1 (n_chunks <= 2 * BLOCK)
    unsigned lm[2] = {0, 0}, tm[2] = {0, 0}, am[2] = {0, 0};
    for (int i = 0; i < 2; ++i)
        if (2 * tid + i < n_chunks) { lm[i] = sm.less_mask[2 * tid + i]; tm[i] = sm.tie_mask[2 * tid + i]; }
    int scan_total;
    int tie_rank = block_excl_scan<BLOCK>(__popc(tm[0]) + __popc(tm[1]), &scan_total, sm.warp_sums);
    for (int i = 0; i < 2; ++i) {
        const int c = 2 * tid + i;
        if (c < n_chunks) {
            // the first (t_c - tie_rank) ties of the chunk are cached
            unsigned tie_cached = 0, rest = tm[i];
            for (int left = t_c - tie_rank; left > 0 && rest != 0; --left) { tie_cached |= rest & (0u - rest); rest &= rest - 1u; }
            const unsigned valid = 32 * c + 32 <= g ? 0xffffffffu : ((1u << (g - 32 * c)) - 1u);
            am[i] = ~(lm[i] | tie_cached) & valid;
            tie_rank += __popc(tm[i]);
        }
    }
    int pos = block_excl_scan<BLOCK>(__popc(am[0]) + __popc(am[1]), &scan_total, sm.warp_sums);
    for (int i = 0; i < 2; ++i)
        if (2 * tid + i < n_chunks) {
            sm.less_mask[2 * tid + i] = am[i];
            sm.chunk_pos[2 * tid + i] = pos;
            pos += __popc(am[i]);
        }
    __syncthreads();
    const unsigned lt = (1u << lane) - 1u;
    for (int c = warp; c < n_chunks; c += WARPS) {
        const unsigned a = sm.less_mask[c];
        const int e = 32 * c + lane;
        const bool active = (a >> lane) & 1u;
        if (e < g && COCODIFF_IN_BOUNDS(base + e >= 0 && base + e < p.n, p.debug)) p.mask[base + e] = active ? 1 : 0;
        if (active) {
            const int o = out_base + sm.chunk_pos[c] + __popc(a & lt);
            if (COCODIFF_IN_BOUNDS(o >= 0 && o < p.n, p.debug)) p.idx[o] = base + e;
        }
    }
    if (grp == 0 && tid == 0) *p.n_active = p.n_groups * (g - p.n_cached);
    __syncthreads();
}

// The same rule for groups of any size: nothing is kept between the passes, the
// metrics are read and compared in each of them.
template <int BLOCK>
__device__ void emit_selection(const SelectParams &p, int grp, const unsigned long long *vals, bool none,
                               unsigned long long mstar, int t_c, int *warp_sums) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int WARPS = BLOCK / 32;
    const int g = p.g, base = grp * g, out_base = grp * (g - p.n_cached);
    const int per_warp = ((g + WARPS - 1) / WARPS + 31) / 32 * 32;
    const int w_lo = warp * per_warp < g ? warp * per_warp : g;
    const int w_hi = w_lo + per_warp < g ? w_lo + per_warp : g;
    const unsigned lt = (1u << lane) - 1u;
    // ties in this warp's range
    int ties = 0;
    if (!none)
        for (int e0 = w_lo; e0 < w_hi; e0 += 32) {
            const int e = e0 + lane;
            ties += __popc(__ballot_sync(0xffffffffu, e < w_hi && vals[e] == mstar));
        }
    int scan_total;
    int tie_rank = block_excl_scan<BLOCK>(lane == 0 ? ties : 0, &scan_total, warp_sums);
    tie_rank = __shfl_sync(0xffffffffu, tie_rank, 0);
    // active units in this warp's range
    int actives = 0;
    {
        int tr = tie_rank;
        for (int e0 = w_lo; e0 < w_hi; e0 += 32) {
            const int e = e0 + lane;
            const unsigned long long v = e < w_hi ? vals[e] : 0ull;
            const bool tie = !none && e < w_hi && v == mstar;
            const unsigned tb = __ballot_sync(0xffffffffu, tie);
            const bool cached = !none && e < w_hi && (v < mstar || (tie && tr + __popc(tb & lt) < t_c));
            actives += __popc(__ballot_sync(0xffffffffu, e < w_hi && !cached));
            tr += __popc(tb);
        }
    }
    int pos = block_excl_scan<BLOCK>(lane == 0 ? actives : 0, &scan_total, warp_sums);
    pos = __shfl_sync(0xffffffffu, pos, 0);
    for (int e0 = w_lo; e0 < w_hi; e0 += 32) {
        const int e = e0 + lane;
        const unsigned long long v = e < w_hi ? vals[e] : 0ull;
        const bool tie = !none && e < w_hi && v == mstar;
        const unsigned tb = __ballot_sync(0xffffffffu, tie);
        const bool cached = !none && e < w_hi && (v < mstar || (tie && tie_rank + __popc(tb & lt) < t_c));
        const bool active = e < w_hi && !cached;
        const unsigned ab = __ballot_sync(0xffffffffu, active);
        if (e < w_hi && COCODIFF_IN_BOUNDS(base + e >= 0 && base + e < p.n, p.debug)) p.mask[base + e] = cached ? 0 : 1;
        if (active) {
            const int o = out_base + pos + __popc(ab & lt);
            if (COCODIFF_IN_BOUNDS(o >= 0 && o < p.n, p.debug)) p.idx[o] = base + e;
        }
        tie_rank += __popc(tb);
        pos += __popc(ab);
    }
    if (grp == 0 && tid == 0) *p.n_active = p.n_groups * (g - p.n_cached);
    __syncthreads();
}

// dyn: the histogram words are ZERO on entry when n_cached != 0 and g <= 65535.
template <int BLOCK>
__device__ void select_group_large(const SelectParams &p, int grp, LargeSel &sm, unsigned *dyn, const int mb) {
    const int tid = threadIdx.x, lane = tid & 31;
    const int g = p.g, n_cached = p.n_cached;
    const bool none = n_cached == 0;
    // the group's metrics; pieces are summed once and kept in metric_out
    const unsigned long long *vals;
    if (p.parts == 0) vals = p.metric + (long long)grp * g;
    else {
        for (int e = tid; e < g; e += BLOCK) p.metric_out[(long long)grp * g + e] = unit_metric(p, grp * g + e);
        __threadfence();
        __syncthreads();  // this block reads back (from the L2) only what it wrote itself
        vals = p.metric_out + (long long)grp * g;
    }
    const bool keyed = g <= 65535;
    const int hist_words = (int)(large_hist_bytes(mb) / 4);
    unsigned short *keys = reinterpret_cast<unsigned short *>(dyn + hist_words);
    unsigned bin = 0;
    if (!none) {
        int *warp_hist = reinterpret_cast<int *>(dyn);
        const int k = n_cached - 1;
        if (keyed) {
            // one pass over the metrics (sixteen loads in flight per thread): keys and their
            // histogram (dyn[0 .. hist_words) is zero on entry)
            constexpr int UL = 16;
            unsigned long long v[UL];
#pragma unroll
            for (int u = 0; u < UL; ++u) v[u] = tid + u * BLOCK < g ? __ldcg(vals + tid + u * BLOCK) : 0ull;
            __syncthreads();  // the histogram was cleared by the caller, before it waited for the metrics
            for (int e0 = tid; e0 < g; e0 += UL * BLOCK) {
                if (e0 != tid) {
#pragma unroll
                    for (int u = 0; u < UL; ++u) v[u] = e0 + u * BLOCK < g ? __ldcg(vals + e0 + u * BLOCK) : 0ull;
                }
#pragma unroll
                for (int u = 0; u < UL; ++u)
                    if (e0 + u * BLOCK < g) {
                        const unsigned key = key_of(v[u], mb);
                        keys[e0 + u * BLOCK] = (unsigned short)key;
                        atomicAdd(&dyn[key >> 1], (key & 1u) ? 0x10000u : 1u);
                    }
            }
            __syncthreads();
            // every thread owns a run of consecutive keys (read in a rotated order: consecutive
            // lanes then touch different banks)
            const int wpt = hist_words / BLOCK;  // words per thread: 8, 16 or 32
            unsigned cnt = 0;
            for (int i = 0; i < wpt; ++i) {
                const unsigned w = dyn[tid * wpt + ((i + tid) & (wpt - 1))];
                cnt += (w & 0xffffu) + (w >> 16);
            }
            int total;
            const int excl = block_excl_scan<BLOCK>((int)cnt, &total, sm.warp_sums);
            if (cnt > 0 && excl <= k && k < excl + (int)cnt) { sm.sel_owner = tid; sm.sel_k = k - excl; }
            __syncthreads();
            // the first warp walks the winning thread's run: lane l takes word l
            if (tid < 32) {
                const int owner = sm.sel_owner, kk0 = sm.sel_k;
                __syncwarp();
                const unsigned w = lane < wpt ? dyn[owner * wpt + lane] : 0u;
                const int lo = (int)(w & 0xffffu), hi = (int)(w >> 16);
                int incl = lo + hi;
#pragma unroll
                for (int off = 1; off < 32; off <<= 1) {
                    const int t = __shfl_up_sync(0xffffffffu, incl, off);
                    if (lane >= off) incl += t;
                }
                const int before = incl - lo - hi;
                if (before <= kk0 && kk0 < incl) {
                    const bool in_hi = kk0 >= before + lo;
                    sm.sel_bin = (owner * wpt + lane) * 2 + (in_hi ? 1 : 0);
                    sm.sel_k = kk0 - before - (in_hi ? lo : 0);
                    sm.n_cand = in_hi ? hi : lo;
                }
            }
            __syncthreads();
            bin = (unsigned)sm.sel_bin;
            const int kk = sm.sel_k, n_cand = sm.n_cand;
            const int low_bits = key_low_bits(bin, mb);
            __syncthreads();
            if (low_bits == 0) {
                if (tid == 0) { sm.mstar = key_base(bin, mb); sm.t_c = kk + 1; }
            } else if (n_cand <= kCandMax) {
                // the few units of that key: fetched again and ranked by counting
                if (tid == 0) sm.n_cand = 0;
                __syncthreads();
                for (int e = tid; e < g; e += BLOCK)
                    if (keys[e] == bin) {
                        const int slot = atomicAdd(&sm.n_cand, 1);
                        if (slot < kCandMax) { sm.cand_val[slot] = __ldcg(vals + e); sm.cand_idx[slot] = e; }
                    }
                __syncthreads();
                for (int i = tid; i < n_cand; i += BLOCK) {
                    const unsigned long long my = sm.cand_val[i];
                    const int my_e = sm.cand_idx[i];
                    int rank = 0, ties_before = 0;
                    for (int j = 0; j < n_cand; ++j) {
                        const unsigned long long o = sm.cand_val[j];
                        const bool tb = (o == my) & (sm.cand_idx[j] < my_e);
                        rank += (o < my) | tb;
                        ties_before += tb;
                    }
                    if (rank == kk) { sm.mstar = my; sm.t_c = ties_before + 1; }
                }
            } else {
                // many units of that key: radix passes over the bits below the key
                unsigned long long prefix;
                int k_eq;
                radix_passes<BLOCK>(vals, keys, g, bin, 8 * ((low_bits - 1) / 8), kk, sm, warp_hist, &prefix, &k_eq);
                if (tid == 0) {
                    const int covered = 8 * ((low_bits - 1) / 8) + 8;
                    const unsigned long long lowmask = covered >= 64 ? ~0ull : ((1ull << covered) - 1ull);
                    sm.mstar = (key_base(bin, mb) & ~lowmask) | prefix;
                    sm.t_c = k_eq + 1;
                }
            }
        } else {
            unsigned long long mx = 0;
            for (int e = tid; e < g; e += BLOCK) { const unsigned long long v = __ldcg(vals + e); mx = v > mx ? v : mx; }
            mx = block_max_u64<BLOCK>(mx, sm.slots);
            int top = 56;
            while (top > 0 && (mx >> top) == 0ull) top -= 8;
            unsigned long long prefix;
            int k_eq;
            radix_passes<BLOCK>(vals, nullptr, g, 0u, top, k, sm, warp_hist, &prefix, &k_eq);
            if (tid == 0) { sm.mstar = prefix; sm.t_c = k_eq + 1; }
        }
    }
    __syncthreads();
    if (keyed) emit_selection_masks<BLOCK>(p, grp, vals, keys, bin, none, none ? 0ull : sm.mstar, none ? 0 : sm.t_c, sm);
    else emit_selection<BLOCK>(p, grp, vals, none, none ? 0ull : sm.mstar, none ? 0 : sm.t_c, sm.warp_sums);
}

// ---------------------------------------------------------------------------
// fix(|a - b|): one fp32 subtraction, scale by 2^16, truncate, saturate to 32
// bits; NaN counts as the saturated value.
__device__ __forceinline__ unsigned fix16(float a, float b) {
    const float d = fabsf(a - b);
    const unsigned r = __float2uint_rz(d * 65536.0f);  // saturating conversion
    return d != d ? 0xffffffffu : r;
}

__device__ __forceinline__ unsigned long long l1_of_vec_exact(const uint4 a, const uint4 b) {
    const unsigned aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    unsigned long long s = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        s += fix16(__uint_as_float(aw[q] << 16), __uint_as_float(bw[q] << 16));
        s += fix16(__uint_as_float(aw[q] & 0xffff0000u), __uint_as_float(bw[q] & 0xffff0000u));
    }
    return s;
}

// The same sum without a float-to-integer conversion per element: for
// |d| * 2^16 < 2^23 the fused multiply-add |d| * 2^16 + 2^23, rounded toward
// zero, has the truncated value in its mantissa bits (the product is exact and
// the spacing of floats in [2^23, 2^24) is 1).  A larger difference, Inf or NaN
// shows as a bit pattern >= that of 2^24; such a vector is redone exactly.
__device__ __forceinline__ unsigned long long l1_of_vec(const uint4 a, const uint4 b) {
    const unsigned aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
    unsigned s = 0, top = 0;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        const float dl = __uint_as_float(aw[q] << 16) - __uint_as_float(bw[q] << 16);
        const float dh = __uint_as_float(aw[q] & 0xffff0000u) - __uint_as_float(bw[q] & 0xffff0000u);
        const unsigned ul = __float_as_uint(__fmaf_rz(fabsf(dl), 65536.0f, 8388608.0f));
        const unsigned uh = __float_as_uint(__fmaf_rz(fabsf(dh), 65536.0f, 8388608.0f));
        s += ul + uh;
        top = max(top, max(ul, uh));
    }
    if (top >= 0x4B800000u) return l1_of_vec_exact(a, b);
    return (unsigned long long)(s - 8u * 0x4B000000u);  // eight biases of 2^23, modulo 2^32
}

// Sum over vectors [v0, v1) of one unit, `stride` threads apart starting at
// v0 + first; U loads of each tensor are in flight per thread.
__device__ __forceinline__ unsigned long long metric_span(const MetricParams &p, const long long unit_base,
                                                          const long long v0, const long long v1, const int first,
                                                          const int stride) {
    constexpr int U = kMetricUnroll;
    const uint4 *pc = p.cur + unit_base, *pp = p.prev + unit_base;
    const long long limit = (long long)p.n_units * p.unit_vecs;
    (void)limit;
    unsigned long long acc = 0;
    for (long long v = v0 + first; v < v1; v += (long long)stride * U) {
        uint4 a[U], b[U];
#pragma unroll
        for (int i = 0; i < U; ++i)
            if (v + (long long)stride * i < v1) {
                const bool ok = COCODIFF_IN_BOUNDS(unit_base + v + (long long)stride * i < limit, p.debug);
                // cur_v is read again by the compaction of the active units: keep it in the L2;
                // prev_v is not: evict first
                a[i] = ok ? __ldg(pc + v + (long long)stride * i) : make_uint4(0, 0, 0, 0);
                b[i] = ok ? __ldcs(pp + v + (long long)stride * i) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
        for (int i = 0; i < U; ++i)
            if (v + (long long)stride * i < v1) acc += l1_of_vec(a[i], b[i]);
    }
    return acc;
}

}  // namespace vmajor
}  // namespace cocodiff

// C ABI of libcocodiff: argument validation, stream / event wiring and the
// launch plan of every entry point declared in include/cocodiff.h.  No kernel
// lives here and no device memory is allocated here.
#include <cmath>
#include <cstring>
#include <mutex>

#include "../../include/cocodiff.h"
#include "common.cuh"

using namespace cocodiff;

namespace {

thread_local int g_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
    g_last_cuda_error = (int)e;
    return COCODIFF_CUDA_ERROR;
}

#define CK(expr)                                       \
    do {                                               \
        const cudaError_t e__ = (expr);                \
        if (e__ != cudaSuccess) return cuda_fail(e__); \
    } while (0)

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

bool overlap(const void *a, size_t na, const void *b, size_t nb) {
    if (!a || !b || na == 0 || nb == 0) return false;
    const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
    return x < y + nb && y < x + na;
}

// a row is D/8 16-byte vectors, at most one per lane of a warp
bool supported_d(int D) { return D >= 8 && D <= 256 && D % 8 == 0; }

int check_shape(int P, int S, int H, int D) {
    if (P < 1 || S < 0 || H < 1) return COCODIFF_INVALID_ARG;
    if (!supported_d(D)) return COCODIFF_BAD_SHAPE;
    if (S % P != 0 || H % P != 0 || P > H) return COCODIFF_BAD_SHAPE;
    if ((long long)S * H * D > (1LL << 40)) return COCODIFF_BAD_SHAPE;
    return COCODIFF_OK;
}

int check_unit(int P, int S, int T) {
    if (T < 1) return COCODIFF_INVALID_ARG;
    if ((S / P) % T != 0) return COCODIFF_BAD_SHAPE;
    return COCODIFF_OK;
}

// Two timing-less events per (thread, device) for the fork / join of the V stream.
// (They live as long as the thread's use of the device: destroying them from a thread-exit
// hook could run after the runtime has shut down.)
struct ForkJoin {
    cudaEvent_t fork = nullptr, join = nullptr;
};
constexpr int kMaxDevices = 64;
thread_local ForkJoin g_events[kMaxDevices];

int get_events(ForkJoin **out) {
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return COCODIFF_INVALID_ARG;
    ForkJoin &fj = g_events[dev];
    if (!fj.fork) {
        CK(cudaEventCreateWithFlags(&fj.fork, cudaEventDisableTiming));
        CK(cudaEventCreateWithFlags(&fj.join, cudaEventDisableTiming));
    }
    *out = &fj;
    return COCODIFF_OK;
}

int join_streams(ForkJoin *fj, cudaStream_t sq, cudaStream_t sv) {
    CK(cudaEventRecord(fj->join, sv));
    CK(cudaStreamWaitEvent(sq, fj->join, 0));
    return COCODIFF_OK;
}

// Bounds-checked build: one violation counter per device, inside the library image.
#ifdef COCODIFF_DEBUG_BOUNDS
static __device__ unsigned long long g_bounds_violations;
unsigned long long *debug_counter() {
    static std::mutex mu;
    static unsigned long long *addr[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void *ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_bounds_violations) != cudaSuccess) return nullptr;
        addr[dev] = static_cast<unsigned long long *>(ptr);
    }
    return addr[dev];
}
#else
unsigned long long *debug_counter() { return nullptr; }
#endif

// Extents (in elements / floats) of the buffers a move touches, for the bounds-checked build.
void set_extents(MoveParams &p, long long src, long long dst, long long cs) {
    p.src_extent = src;
    p.dst_extent = dst;
    p.cs_extent = cs;
    p.debug = debug_counter();
}

MoveParams seq_to_head(int S, int H, int D) {
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = S;
    p.H = H;
    p.D = D;
    p.src_tok = (long long)H * D;
    p.src_head = D;
    p.dst_tok = D;
    p.dst_head = (long long)S * D;
    p.map = MAP_FULL;
    p.T = 1;
    set_extents(p, (long long)S * H * D, (long long)S * H * D, (long long)S * D);
    return p;
}

// Shared by cocodiff_ulysses_a2a (no weights) and cocodiff_prologue.
// A call's first kernel is launched with the programmatic attribute and waits for its
// predecessor in the stream before it touches memory; its last kernel lets whatever follows
// become resident while it drains.  Consecutive calls on one stream (layer after layer) then
// overlap launch latency, ramp-up and drain without giving up their order; a successor that
// was launched without the attribute starts when the last kernel has completed, as ever.
constexpr int kChainedLaunch = PDL_LAUNCH_ATTR | PDL_WAIT_AT_START | PDL_TRIGGER;

int exchange(const uint16_t *q, const uint16_t *k, const uint16_t *v, uint16_t *qh, uint16_t *kh,
             uint16_t *vh, const uint16_t *wq, const uint16_t *wk, float eps, const float *cs, int S,
             int H, int D, int order, cudaStream_t sq, cudaStream_t sv) {
    MoveParams base = seq_to_head(S, H, D);
    base.cs = cs;
    base.eps = eps;
    const bool two_streams = order == COCODIFF_V_FIRST && sv != sq && v != nullptr && (q || k);
    if (order == COCODIFF_V_FIRST && sv == sq && v != nullptr && (q || k)) {
        // V first on one stream: V's launch, then Q/K's launch with the programmatic attribute.
        // Q/K's grid does not read V's output, so it starts while V's last blocks drain, and
        // waits for V's grid only before it completes (the stream's order of completion holds).
        MoveParams pv = base;
        pv.job[pv.njobs++] = MoveJob{v, vh, nullptr, nullptr};
        pv.pdl = kChainedLaunch;  // Q/K's launch follows once V's blocks have passed their wait
        MoveParams pqk = base;
        if (q) pqk.job[pqk.njobs++] = MoveJob{q, qh, wq, nullptr};
        if (k) pqk.job[pqk.njobs++] = MoveJob{k, kh, wk, nullptr};
        pqk.pdl = PDL_LAUNCH_ATTR | PDL_WAIT_AT_END | PDL_TRIGGER;
        CK(launch_move(pv, sq));
        CK(launch_move(pqk, sq));
        return COCODIFF_OK;
    }
    if (order == COCODIFF_LUMP || !two_streams) {
        // one launch; V's blocks come first in the grid
        MoveParams p = base;
        if (v) p.job[p.njobs++] = MoveJob{v, vh, nullptr, nullptr};
        if (q) p.job[p.njobs++] = MoveJob{q, qh, wq, nullptr};
        if (k) p.job[p.njobs++] = MoveJob{k, kh, wk, nullptr};
        if (p.njobs == 0) return COCODIFF_OK;
        p.pdl = kChainedLaunch;
        CK(launch_move(p, sq));
        return COCODIFF_OK;
    }
    ForkJoin *fj = nullptr;
    const int rc = get_events(&fj);
    if (rc != COCODIFF_OK) return rc;
    CK(cudaEventRecord(fj->fork, sq));
    CK(cudaStreamWaitEvent(sv, fj->fork, 0));
    MoveParams pv = base;
    pv.job[pv.njobs++] = MoveJob{v, vh, nullptr, nullptr};
    MoveParams pqk = base;
    if (q) pqk.job[pqk.njobs++] = MoveJob{q, qh, wq, nullptr};
    if (k) pqk.job[pqk.njobs++] = MoveJob{k, kh, wk, nullptr};
    cudaError_t e = launch_move(pv, sv);
    if (e == cudaSuccess) e = launch_move(pqk, sq);
    // whatever happened, stream_qk is ordered behind stream_v again
    const int rj = join_streams(fj, sq, sv);
    if (e != cudaSuccess) return cuda_fail(e);
    return rj;
}

int check_pairs(const uint16_t *const in[3], uint16_t *const out[3], size_t bytes) {
    for (int i = 0; i < 3; ++i) {
        if ((in[i] == nullptr) != (out[i] == nullptr)) return COCODIFF_INVALID_ARG;
        if (!aligned16(in[i]) || !aligned16(out[i])) return COCODIFF_MISALIGNED;
    }
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) {
            if (overlap(in[i], bytes, out[j], bytes)) return COCODIFF_ALIASING;
            if (i < j && overlap(out[i], bytes, out[j], bytes)) return COCODIFF_ALIASING;
        }
    return COCODIFF_OK;
}


// ---- V-Major helpers --------------------------------------------------------
// Scratch of the metric pass: one 64-bit sum per piece of a unit (see plan_metric),
// plus a spare 256 bytes.  Units that are not cut (parts == 1) need no scratch: their
// sums go straight to the caller's metric array.
size_t vmajor_ws_bytes(int S, int H, int D, int T) {
    const long long n = S / T;
    const MetricPlan pl = plan_metric((int)n, (long long)T * H * D / 8);
    return (((size_t)n * pl.parts * 8 + 255) / 256) * 256 + 256;
}

// Token slots that the selection rule leaves active: (n - n_groups * floor(r * g)) * T.
int active_slots(int S, int T, double r, int n_groups) {
    const int n = S / T, g = n / n_groups;
    return (n - n_groups * (int)std::floor(r * (double)g)) * T;
}

int check_select(const uint16_t *prev_v, const uint16_t *cur_v, int P, int S, int H, int D, int T, double r,
                 int n_groups, const uint64_t *metric, const uint8_t *mask, const int32_t *idx,
                 const int32_t *n_active, const void *workspace, size_t workspace_bytes) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    rc = check_unit(P, S, T);
    if (rc) return rc;
    if (!prev_v || !cur_v || !metric || !mask || !idx || !n_active || !workspace || n_groups < 1 ||
        !(r >= 0.0 && r <= 1.0))
        return COCODIFF_INVALID_ARG;
    if ((S / T) % n_groups != 0) return COCODIFF_BAD_SHAPE;
    if (!aligned16(prev_v) || !aligned16(cur_v) || (reinterpret_cast<uintptr_t>(workspace) & 255u) ||
        (reinterpret_cast<uintptr_t>(metric) & 7u) || (reinterpret_cast<uintptr_t>(idx) & 3u) ||
        (reinterpret_cast<uintptr_t>(n_active) & 3u))
        return COCODIFF_MISALIGNED;
    if (workspace_bytes < vmajor_ws_bytes(S, H, D, T)) return COCODIFF_WORKSPACE_TOO_SMALL;
    return COCODIFF_OK;
}

// in/out pairs of a compaction or scatter: both or neither, aligned, disjoint.
int check_tiles(const uint16_t *const in[3], uint16_t *const out[3], int S, int H, int D, const int32_t *idx,
                const int32_t *n_active) {
    if (!idx || !n_active) return COCODIFF_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(n_active) & 3u))
        return COCODIFF_MISALIGNED;
    return check_pairs(in, out, (size_t)S * H * D * 2);
}

SelectParams make_select_params(const unsigned long long *metric, int n, double r, int n_groups, uint8_t *mask,
                                int32_t *idx, int32_t *n_active) {
    SelectParams sp;
    std::memset(&sp, 0, sizeof sp);
    sp.metric = metric;
    sp.n = n;
    sp.n_groups = n_groups;
    sp.g = n / n_groups;
    sp.n_cached = (int)std::floor(r * (double)sp.g);
    sp.mask = mask;
    sp.idx = idx;
    sp.n_active = n_active;
    sp.debug = debug_counter();
    return sp;
}

// The metric pass and the selection that follows it.
struct SelectionPlan {
    MetricParams mp;
    SelectParams sp;
    bool in_consumer;  // few units: every block of the consuming kernel selects for itself
};

SelectionPlan plan_selection(const uint16_t *prev_v, const uint16_t *cur_v, int S, int H, int D, int T, double r,
                             int n_groups, uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                             void *workspace) {
    const int n = S / T;
    SelectionPlan pl;
    std::memset(&pl.mp, 0, sizeof pl.mp);
    const MetricPlan cut = plan_metric(n, (long long)T * H * D / 8);
    pl.mp.prev = reinterpret_cast<const uint4 *>(prev_v);
    pl.mp.cur = reinterpret_cast<const uint4 *>(cur_v);
    pl.mp.unit_vecs = (long long)T * H * D / 8;
    pl.mp.part_vecs = cut.part_vecs;
    pl.mp.parts = cut.parts;
    pl.mp.warp_mode = cut.warp_mode;
    pl.mp.n_units = n;
    pl.mp.debug = debug_counter();
    pl.sp = make_select_params(reinterpret_cast<const unsigned long long *>(metric), n, r, n_groups, mask, idx,
                               n_active);
    if (cut.parts == 1) {
        pl.mp.out = reinterpret_cast<unsigned long long *>(metric);  // whole units: the sums are the metric
    } else {
        pl.mp.out = reinterpret_cast<unsigned long long *>(workspace);
        pl.sp.metric = nullptr;
        pl.sp.partial = pl.mp.out;
        pl.sp.metric_out = reinterpret_cast<unsigned long long *>(metric);
        pl.sp.parts = cut.parts;
    }
    pl.in_consumer = n > 0 && n <= kCountMax;
    return pl;
}

// Compaction of up to three tensors in one launch; slot order (Q, K, V), V's blocks first.
// cache[i], when given, also receives the rows (the receiver-side scatter in the same pass).
// direct: there is no compact buffer; the rows go to their slots of cache[i] only.
MoveParams make_pack_params(const uint16_t *const in[3], uint16_t *const out[3], uint16_t *const cache[3],
                            const uint16_t *wq, const uint16_t *wk, float eps, const float *cs, const int32_t *idx,
                            const int32_t *n_active, int slots, int S, int H, int D, int T, bool direct = false) {
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = slots;
    p.H = H;
    p.D = D;
    p.src_tok = (long long)H * D;
    p.src_head = D;
    p.dst_tok = D;
    p.dst_head = COMPACT_STRIDE;
    p.dst2_tok = D;
    p.dst2_head = (long long)S * D;
    p.map = MAP_GATHER;
    p.T = T;
    p.n_units = S / T;
    p.idx = idx;
    p.n_active = n_active;
    p.cs = cs;
    p.eps = eps;
    set_extents(p, (long long)S * H * D, (long long)S * H * D, (long long)S * D);
    p.dst2_extent = (long long)S * H * D;
    if (direct) {
        p.map = MAP_ACTIVE;
        p.dst_head = (long long)S * D;
        if (in[2]) p.job[p.njobs++] = MoveJob{in[2], cache[2], nullptr, nullptr};
        if (in[0]) p.job[p.njobs++] = MoveJob{in[0], cache[0], wq, nullptr};
        if (in[1]) p.job[p.njobs++] = MoveJob{in[1], cache[1], wk, nullptr};
        return p;
    }
    if (in[2]) p.job[p.njobs++] = MoveJob{in[2], out[2], nullptr, cache ? cache[2] : nullptr};
    if (in[0]) p.job[p.njobs++] = MoveJob{in[0], out[0], wq, cache ? cache[0] : nullptr};
    if (in[1]) p.job[p.njobs++] = MoveJob{in[1], out[1], wk, cache ? cache[1] : nullptr};
    return p;
}

int enqueue_pack(const uint16_t *const in[3], uint16_t *const out[3], const uint16_t *wq, const uint16_t *wk,
                 float eps, const float *cs, const int32_t *idx, const int32_t *n_active, int slots, int S,
                 int H, int D, int T, cudaStream_t st) {
    MoveParams p = make_pack_params(in, out, nullptr, wq, wk, eps, cs, idx, n_active, slots, S, H, D, T);
    if (p.njobs == 0) return COCODIFF_OK;
    p.pdl = kChainedLaunch;
    CK(launch_selective_move(p, nullptr, st));  // a resident wave that walks the active tiles only
    return COCODIFF_OK;
}

// Metric, selection and the compaction (+ scatter) of the given tensors on one stream,
// chained with programmatic dependent launches.
int enqueue_select_and_pack(const SelectionPlan &pl, const uint16_t *const in[3], uint16_t *const out[3],
                            uint16_t *const cache[3], const uint16_t *wq, const uint16_t *wk, float eps,
                            const float *cs, int slots, int S, int H, int D, int T, cudaStream_t st,
                            bool direct = false) {
    MoveParams p =
        make_pack_params(in, out, cache, wq, wk, eps, cs, pl.sp.idx, pl.sp.n_active, slots, S, H, D, T, direct);
    p.slots_exact = 1;  // slots = (n - n_groups * floor(r * g)) * T, what the selection will publish
    // the consuming kernel selects for itself when it has few units to rank and at least one block
    const bool consume = p.njobs > 0 && pl.in_consumer && slots > 0;
    MetricParams mp = pl.mp;
    mp.pdl = kChainedLaunch;  // the trigger follows the block's loads
    CK(launch_metric(mp, st));
    if (!consume)  // a selection launch: many units, or nothing follows that could select for itself
        CK(launch_select(pl.sp, st, pl.mp.n_units > 0 ? (PDL_LAUNCH_ATTR | PDL_WAIT_AT_START | PDL_TRIGGER) : 0));
    if (p.njobs == 0) return COCODIFF_OK;
    p.pdl = pl.mp.n_units > 0 ? kChainedLaunch : 0;
    CK(launch_selective_move(p, consume ? &pl.sp : nullptr, st));
    return COCODIFF_OK;
}

MoveParams make_unpack_params(const uint16_t *const in[3], uint16_t *const out[3], const int32_t *idx,
                              const int32_t *n_active, int slots, int S, int H, int D, int T) {
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = slots;
    p.H = H;
    p.D = D;
    p.src_tok = D;
    p.src_head = COMPACT_STRIDE;
    p.dst_tok = D;
    p.dst_head = (long long)S * D;
    p.map = MAP_SCATTER;
    p.T = T;
    p.n_units = S / T;
    p.idx = idx;
    p.n_active = n_active;
    set_extents(p, (long long)S * H * D, (long long)S * H * D, 0);
    for (int i = 2; i >= 0; --i)
        if (in[i]) p.job[p.njobs++] = MoveJob{in[i], out[i], nullptr, nullptr};
    return p;
}

int enqueue_unpack(const uint16_t *const in[3], uint16_t *const out[3], const int32_t *idx,
                   const int32_t *n_active, int slots, int S, int H, int D, int T, cudaStream_t st) {
    MoveParams p = make_unpack_params(in, out, idx, n_active, slots, S, H, D, T);
    if (p.njobs == 0) return COCODIFF_OK;
    p.pdl = kChainedLaunch;
    CK(launch_selective_move(p, nullptr, st));  // a resident wave that walks the active tiles only
    return COCODIFF_OK;
}

}  // namespace

extern "C" {

const char *cocodiff_status_string(int status) {
    switch (status) {
        case COCODIFF_OK: return "ok";
        case COCODIFF_INVALID_ARG: return "invalid argument";
        case COCODIFF_BAD_SHAPE: return "unsupported shape";
        case COCODIFF_MISALIGNED: return "pointer not 16-byte aligned";
        case COCODIFF_WORKSPACE_TOO_SMALL: return "workspace too small";
        case COCODIFF_CUDA_ERROR: return "CUDA error";
        case COCODIFF_ALIASING: return "input and output overlap";
        default: return "unknown status";
    }
}

int cocodiff_version(void) { return 100; }

int cocodiff_last_cuda_error(void) { return g_last_cuda_error; }

int cocodiff_rope_table_2d(float *cs, const int32_t *pos, int S, int D, double theta, void *stream) {
    if (!cs || !pos || S < 0 || !(theta > 0.0)) return COCODIFF_INVALID_ARG;
    if (!supported_d(D)) return COCODIFF_BAD_SHAPE;
    if (!aligned16(cs) || (reinterpret_cast<uintptr_t>(pos) & 3u)) return COCODIFF_MISALIGNED;
    CK(launch_rope_table(cs, pos, S, D, theta, (cudaStream_t)stream));
    return COCODIFF_OK;
}

int cocodiff_qk_norm_rope(const uint16_t *q, const uint16_t *k, uint16_t *q_out, uint16_t *k_out,
                          const uint16_t *wq, const uint16_t *wk, float eps, const float *cs, int S,
                          int H, int D, void *stream) {
    if (S < 0 || H < 1 || !(eps >= 0.f)) return COCODIFF_INVALID_ARG;
    if (!supported_d(D) || (long long)S * H * D > (1LL << 40)) return COCODIFF_BAD_SHAPE;
    if ((q == nullptr) != (q_out == nullptr) || (k == nullptr) != (k_out == nullptr)) return COCODIFF_INVALID_ARG;
    if ((q && !wq) || (k && !wk)) return COCODIFF_INVALID_ARG;
    if (!aligned16(q) || !aligned16(k) || !aligned16(q_out) || !aligned16(k_out) || !aligned16(wq) ||
        !aligned16(wk) || !aligned16(cs))
        return COCODIFF_MISALIGNED;
    const size_t bytes = (size_t)S * H * D * 2;
    if ((q_out != q && overlap(q, bytes, q_out, bytes)) || (k_out != k && overlap(k, bytes, k_out, bytes)) ||
        overlap(q, bytes, k_out, bytes) || overlap(k, bytes, q_out, bytes) || overlap(q_out, bytes, k_out, bytes))
        return COCODIFF_ALIASING;
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = S;
    p.H = H;
    p.D = D;
    p.src_tok = p.dst_tok = (long long)H * D;
    p.src_head = p.dst_head = D;
    p.map = MAP_FULL;
    p.T = 1;
    p.cs = cs;
    p.eps = eps;
    set_extents(p, (long long)S * H * D, (long long)S * H * D, (long long)S * D);
    if (q) p.job[p.njobs++] = MoveJob{q, q_out, wq};
    if (k) p.job[p.njobs++] = MoveJob{k, k_out, wk};
    if (p.njobs == 0) return COCODIFF_OK;
    p.pdl = kChainedLaunch;
    CK(launch_move(p, (cudaStream_t)stream));
    return COCODIFF_OK;
}

int cocodiff_ulysses_a2a(const uint16_t *q, const uint16_t *k, const uint16_t *v, uint16_t *q_head,
                         uint16_t *k_head, uint16_t *v_head, int P, int S, int H, int D,
                         cocodiff_order order, void *stream_qk, void *stream_v) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    if (order != COCODIFF_LUMP && order != COCODIFF_V_FIRST) return COCODIFF_INVALID_ARG;
    const uint16_t *in[3] = {q, k, v};
    uint16_t *out[3] = {q_head, k_head, v_head};
    rc = check_pairs(in, out, (size_t)S * H * D * 2);
    if (rc) return rc;
    return exchange(q, k, v, q_head, k_head, v_head, nullptr, nullptr, 0.f, nullptr, S, H, D, order,
                    (cudaStream_t)stream_qk, (cudaStream_t)stream_v);
}

int cocodiff_ulysses_a2a_inverse(const uint16_t *q_head, const uint16_t *k_head, const uint16_t *v_head,
                                 uint16_t *q, uint16_t *k, uint16_t *v, int P, int S, int H, int D,
                                 void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    const uint16_t *in[3] = {q_head, k_head, v_head};
    uint16_t *out[3] = {q, k, v};
    rc = check_pairs(in, out, (size_t)S * H * D * 2);
    if (rc) return rc;
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = S;
    p.H = H;
    p.D = D;
    p.src_tok = D;
    p.src_head = (long long)S * D;
    p.dst_tok = (long long)H * D;
    p.dst_head = D;
    p.map = MAP_FULL;
    p.T = 1;
    set_extents(p, (long long)S * H * D, (long long)S * H * D, 0);
    for (int i = 2; i >= 0; --i)
        if (in[i]) p.job[p.njobs++] = MoveJob{in[i], out[i], nullptr};
    if (p.njobs == 0) return COCODIFF_OK;
    p.pdl = kChainedLaunch;
    CK(launch_move(p, (cudaStream_t)stream));
    return COCODIFF_OK;
}

int cocodiff_prologue(const uint16_t *q, const uint16_t *k, const uint16_t *v, uint16_t *q_head,
                      uint16_t *k_head, uint16_t *v_head, const uint16_t *wq, const uint16_t *wk,
                      float eps, const float *cs, int P, int S, int H, int D, cocodiff_order order,
                      void *stream_qk, void *stream_v) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    if (order != COCODIFF_LUMP && order != COCODIFF_V_FIRST) return COCODIFF_INVALID_ARG;
    if ((q && !wq) || (k && !wk) || ((q || k) && !cs) || !(eps >= 0.f)) return COCODIFF_INVALID_ARG;
    if (!aligned16(wq) || !aligned16(wk) || !aligned16(cs)) return COCODIFF_MISALIGNED;
    const uint16_t *in[3] = {q, k, v};
    uint16_t *out[3] = {q_head, k_head, v_head};
    rc = check_pairs(in, out, (size_t)S * H * D * 2);
    if (rc) return rc;
    return exchange(q, k, v, q_head, k_head, v_head, wq, wk, eps, cs, S, H, D, order,
                    (cudaStream_t)stream_qk, (cudaStream_t)stream_v);
}

int cocodiff_prologue_host(const uint16_t *q_host, const uint16_t *k_host, const uint16_t *v_host,
                           uint16_t *q_head_host, uint16_t *k_head_host, uint16_t *v_head_host,
                           uint16_t *dev_in, uint16_t *dev_out, const uint16_t *wq, const uint16_t *wk,
                           float eps, const float *cs, int P, int S, int H, int D, cocodiff_order order,
                           void *stream_qk, void *stream_v) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    if (order != COCODIFF_LUMP && order != COCODIFF_V_FIRST) return COCODIFF_INVALID_ARG;
    if (!q_host || !k_host || !v_host || !q_head_host || !k_head_host || !v_head_host || !dev_in ||
        !dev_out || !wq || !wk || !cs || !(eps >= 0.f))
        return COCODIFF_INVALID_ARG;
    if (!aligned16(dev_in) || !aligned16(dev_out) || !aligned16(wq) || !aligned16(wk) || !aligned16(cs))
        return COCODIFF_MISALIGNED;
    const size_t E = (size_t)S * H * D, bytes = E * 2;
    if (overlap(dev_in, 3 * bytes, dev_out, 3 * bytes)) return COCODIFF_ALIASING;
    cudaStream_t sq = (cudaStream_t)stream_qk, sv = (cudaStream_t)stream_v;
    if (order == COCODIFF_LUMP) sv = sq;
    uint16_t *din[3] = {dev_in + 2 * E, dev_in, dev_in + E};      // V, Q, K
    uint16_t *dout[3] = {dev_out + 2 * E, dev_out, dev_out + E};
    const uint16_t *hin[3] = {v_host, q_host, k_host};
    uint16_t *hout[3] = {v_head_host, q_head_host, k_head_host};
    const uint16_t *w[3] = {nullptr, wq, wk};
    ForkJoin *fj = nullptr;
    if (sv != sq) {
        rc = get_events(&fj);
        if (rc) return rc;
        CK(cudaEventRecord(fj->fork, sq));
        CK(cudaStreamWaitEvent(sv, fj->fork, 0));
    }
    // Token chunks alternate between the two streams: while one chunk's results
    // travel back to the host, the next chunk's inputs arrive and its rows are
    // processed.  Inside a chunk V is copied first and its blocks lead the grid.
    const int n_chunks = (sv != sq && S >= 8 * 256) ? 8 : 1;  // 16 chunks measure the same, 24 and 32 slower
    int chunk = (S + n_chunks - 1) / n_chunks;
    chunk = (chunk + 31) / 32 * 32;
    const size_t tok_in = (size_t)H * D, pitch = (size_t)S * D * 2;
    auto run_chunks = [&]() -> cudaError_t {
        cudaError_t e = cudaSuccess;
        for (int c = 0, s0 = 0; s0 < S; ++c, s0 += chunk) {
            const int len = s0 + chunk <= S ? chunk : S - s0;
            cudaStream_t st = (c % 2 == 0) ? sv : sq;
            MoveParams p = seq_to_head(S, H, D);
            p.n_slots = len;
            p.cs = cs + (size_t)s0 * D;
            p.eps = eps;
            set_extents(p, (long long)len * H * D, (long long)E - (long long)s0 * D, (long long)(S - s0) * D);
            for (int i = 0; i < 3; ++i) {
                e = cudaMemcpyAsync(din[i] + s0 * tok_in, hin[i] + s0 * tok_in, (size_t)len * tok_in * 2,
                                    cudaMemcpyHostToDevice, st);
                if (e != cudaSuccess) return e;
                p.job[p.njobs++] = MoveJob{din[i] + s0 * tok_in, dout[i] + (size_t)s0 * D, w[i], nullptr};
            }
            e = launch_move(p, st);
            if (e != cudaSuccess) return e;
            for (int i = 0; i < 3; ++i) {
                e = cudaMemcpy2DAsync(hout[i] + (size_t)s0 * D, pitch, dout[i] + (size_t)s0 * D, pitch,
                                      (size_t)len * D * 2, (size_t)H, cudaMemcpyDeviceToHost, st);
                if (e != cudaSuccess) return e;
            }
        }
        return e;
    };
    const cudaError_t e = run_chunks();
    // whatever happened, stream_qk is ordered behind stream_v again
    if (sv != sq) {
        const int rj = join_streams(fj, sq, sv);
        if (e == cudaSuccess && rj) return rj;
    }
    if (e != cudaSuccess) return cuda_fail(e);
    return COCODIFF_OK;
}

size_t cocodiff_vmajor_workspace_bytes(int P, int S, int H, int D, int T) {
    if (P < 1 || T < 1 || S < 0 || H < 1 || !supported_d(D)) return 0;
    return vmajor_ws_bytes(S, H, D, T);
}

int cocodiff_vmajor_select(const uint64_t *metric, int n, double r, int n_groups, uint8_t *mask,
                           int32_t *idx, int32_t *n_active, void *stream) {
    if (!metric || !mask || !idx || !n_active || n < 0 || n_groups < 1 || !(r >= 0.0 && r <= 1.0))
        return COCODIFF_INVALID_ARG;
    if (n % n_groups != 0) return COCODIFF_BAD_SHAPE;
    if ((reinterpret_cast<uintptr_t>(metric) & 7u) || (reinterpret_cast<uintptr_t>(idx) & 3u) ||
        (reinterpret_cast<uintptr_t>(n_active) & 3u))
        return COCODIFF_MISALIGNED;
    const SelectParams sp = make_select_params(reinterpret_cast<const unsigned long long *>(metric), n, r, n_groups,
                                               mask, idx, n_active);
    CK(launch_select(sp, (cudaStream_t)stream));
    return COCODIFF_OK;
}

int cocodiff_vmajor_select_compact(const uint16_t *prev_v, const uint16_t *cur_v, int P, int S, int H,
                                   int D, int T, double r, int n_groups, uint64_t *metric, uint8_t *mask,
                                   int32_t *idx, int32_t *n_active, uint16_t *v_compact, void *workspace,
                                   size_t workspace_bytes, void *stream) {
    int rc = check_select(prev_v, cur_v, P, S, H, D, T, r, n_groups, metric, mask, idx, n_active, workspace,
                          workspace_bytes);
    if (rc) return rc;
    const uint16_t *in[3] = {nullptr, nullptr, v_compact ? cur_v : nullptr};
    uint16_t *out[3] = {nullptr, nullptr, v_compact};
    if (v_compact) {
        rc = check_tiles(in, out, S, H, D, idx, n_active);
        if (rc) return rc;
        if (overlap(prev_v, (size_t)S * H * D * 2, v_compact, (size_t)S * H * D * 2)) return COCODIFF_ALIASING;
    }
    const SelectionPlan pl = plan_selection(prev_v, cur_v, S, H, D, T, r, n_groups, metric, mask, idx, n_active, workspace);
    // the host knows how many units the rule leaves active: exact grid
    return enqueue_select_and_pack(pl, in, out, nullptr, nullptr, nullptr, 0.f, nullptr, active_slots(S, T, r, n_groups),
                                   S, H, D, T, (cudaStream_t)stream);
}

int cocodiff_pack_active(const uint16_t *x, const uint16_t *w, float eps, const float *cs,
                         const int32_t *idx, const int32_t *n_active, uint16_t *x_compact, int P, int S,
                         int H, int D, int T, void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    rc = check_unit(P, S, T);
    if (rc) return rc;
    if (!x || !x_compact || !(eps >= 0.f)) return COCODIFF_INVALID_ARG;
    if (!aligned16(w) || !aligned16(cs)) return COCODIFF_MISALIGNED;
    // one tensor: it travels in the Q slot when it is normalised, in the V slot otherwise
    const uint16_t *in[3] = {w ? x : nullptr, nullptr, w ? nullptr : x};
    uint16_t *out[3] = {w ? x_compact : nullptr, nullptr, w ? nullptr : x_compact};
    rc = check_tiles(in, out, S, H, D, idx, n_active);
    if (rc) return rc;
    return enqueue_pack(in, out, w, nullptr, eps, cs, idx, n_active, S, S, H, D, T, (cudaStream_t)stream);
}

int cocodiff_pack_active_qkv(const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *wq,
                             const uint16_t *wk, float eps, const float *cs, const int32_t *idx,
                             const int32_t *n_active, uint16_t *q_compact, uint16_t *k_compact,
                             uint16_t *v_compact, int P, int S, int H, int D, int T, void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    rc = check_unit(P, S, T);
    if (rc) return rc;
    if ((q && !wq) || (k && !wk) || !(eps >= 0.f)) return COCODIFF_INVALID_ARG;
    if (!aligned16(wq) || !aligned16(wk) || !aligned16(cs)) return COCODIFF_MISALIGNED;
    const uint16_t *in[3] = {q, k, v};
    uint16_t *out[3] = {q_compact, k_compact, v_compact};
    rc = check_tiles(in, out, S, H, D, idx, n_active);
    if (rc) return rc;
    return enqueue_pack(in, out, wq, wk, eps, cs, idx, n_active, S, S, H, D, T, (cudaStream_t)stream);
}

int cocodiff_unpack(const uint16_t *x_compact, const int32_t *idx, const int32_t *n_active,
                    uint16_t *x_cache, int P, int S, int H, int D, int T, void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    rc = check_unit(P, S, T);
    if (rc) return rc;
    if (!x_compact || !x_cache) return COCODIFF_INVALID_ARG;
    const uint16_t *in[3] = {nullptr, nullptr, x_compact};
    uint16_t *out[3] = {nullptr, nullptr, x_cache};
    rc = check_tiles(in, out, S, H, D, idx, n_active);
    if (rc) return rc;
    return enqueue_unpack(in, out, idx, n_active, S, S, H, D, T, (cudaStream_t)stream);
}

int cocodiff_unpack_qkv(const uint16_t *q_compact, const uint16_t *k_compact, const uint16_t *v_compact,
                        const int32_t *idx, const int32_t *n_active, uint16_t *q_cache, uint16_t *k_cache,
                        uint16_t *v_cache, int P, int S, int H, int D, int T, void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    rc = check_unit(P, S, T);
    if (rc) return rc;
    const uint16_t *in[3] = {q_compact, k_compact, v_compact};
    uint16_t *out[3] = {q_cache, k_cache, v_cache};
    rc = check_tiles(in, out, S, H, D, idx, n_active);
    if (rc) return rc;
    return enqueue_unpack(in, out, idx, n_active, S, S, H, D, T, (cudaStream_t)stream);
}

int cocodiff_selective_prologue(const uint16_t *prev_v, const uint16_t *q, const uint16_t *k,
                                const uint16_t *v, const uint16_t *wq, const uint16_t *wk, float eps,
                                const float *cs, int P, int S, int H, int D, int T, double r, int n_groups,
                                uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                                uint16_t *q_compact, uint16_t *k_compact, uint16_t *v_compact,
                                uint16_t *q_cache, uint16_t *k_cache, uint16_t *v_cache, void *workspace,
                                size_t workspace_bytes, cocodiff_order order, void *stream_qk, void *stream_v) {
    int rc = check_select(prev_v, v, P, S, H, D, T, r, n_groups, metric, mask, idx, n_active, workspace,
                          workspace_bytes);
    if (rc) return rc;
    if (order != COCODIFF_LUMP && order != COCODIFF_V_FIRST) return COCODIFF_INVALID_ARG;
    if (!q || !k || !wq || !wk || !cs || !(eps >= 0.f)) return COCODIFF_INVALID_ARG;
    if (!aligned16(wq) || !aligned16(wk) || !aligned16(cs)) return COCODIFF_MISALIGNED;
    const bool do_unpack = q_cache || k_cache || v_cache;
    if (do_unpack && !(q_cache && k_cache && v_cache)) return COCODIFF_INVALID_ARG;
    // direct delivery: no compact buffers, the active rows go straight to the caches
    const bool direct = !q_compact && !k_compact && !v_compact;
    if (direct ? !do_unpack : !(q_compact && k_compact && v_compact)) return COCODIFF_INVALID_ARG;
    const uint16_t *in[3] = {q, k, v};
    uint16_t *comp[3] = {q_compact, k_compact, v_compact};
    const size_t bytes = (size_t)S * H * D * 2;
    if (!direct) {
        rc = check_tiles(in, comp, S, H, D, idx, n_active);
        if (rc) return rc;
        for (int i = 0; i < 3; ++i)
            if (overlap(prev_v, bytes, comp[i], bytes)) return COCODIFF_ALIASING;
    }
    const uint16_t *comp_in[3] = {q_compact, k_compact, v_compact};
    uint16_t *cache[3] = {q_cache, k_cache, v_cache};
    if (do_unpack) {
        rc = check_tiles(direct ? in : comp_in, cache, S, H, D, idx, n_active);
        if (rc) return rc;
        for (int i = 0; i < 3; ++i)
            for (int j = 0; j < 3; ++j)
                if (overlap(in[i], bytes, cache[j], bytes) || overlap(prev_v, bytes, cache[j], bytes))
                    return COCODIFF_ALIASING;
    }
    // the host knows how many units will be active: grids are sized exactly
    const int slots = active_slots(S, T, r, n_groups);
    cudaStream_t sq = (cudaStream_t)stream_qk, sv = (cudaStream_t)stream_v;
    const SelectionPlan pl = plan_selection(prev_v, v, S, H, D, T, r, n_groups, metric, mask, idx, n_active, workspace);
    uint16_t *const *scatter = do_unpack ? cache : nullptr;
    // One stream: metric pass, (selection,) one compaction + scatter launch for V, Q and K,
    // chained with programmatic dependent launches: each successor becomes resident while
    // its predecessor drains and orders itself with griddepcontrol.wait.
    if (order == COCODIFF_LUMP || sv == sq)
        return enqueue_select_and_pack(pl, in, comp, scatter, wq, wk, eps, cs, slots, S, H, D, T, sq, direct);
    // V first: metric, selection and V's compaction + scatter on stream_v; Q and K follow on
    // stream_qk once V's part is done and read the list that V's part published.
    ForkJoin *fj = nullptr;
    rc = get_events(&fj);
    if (rc) return rc;
    CK(cudaEventRecord(fj->fork, sq));
    CK(cudaStreamWaitEvent(sv, fj->fork, 0));
    const uint16_t *in_v[3] = {nullptr, nullptr, v};
    uint16_t *out_v[3] = {nullptr, nullptr, v_compact};
    uint16_t *cache_v[3] = {nullptr, nullptr, v_cache};
    rc = enqueue_select_and_pack(pl, in_v, out_v, do_unpack ? cache_v : nullptr, nullptr, nullptr, 0.f, nullptr, slots, S, H,
                                 D, T, sv, direct);
    // whatever happened on stream_v, stream_qk is ordered behind it again
    const int rj = join_streams(fj, sq, sv);
    if (rc) return rc;
    if (rj) return rj;
    const uint16_t *in_qk[3] = {q, k, nullptr};
    uint16_t *out_qk[3] = {q_compact, k_compact, nullptr};
    uint16_t *cache_qk[3] = {q_cache, k_cache, nullptr};
    MoveParams p = make_pack_params(in_qk, out_qk, do_unpack ? cache_qk : nullptr, wq, wk, eps, cs, idx, n_active, slots, S,
                                    H, D, T, direct);
    p.slots_exact = 1;
    p.pdl = kChainedLaunch;
    CK(launch_selective_move(p, nullptr, sq));
    return COCODIFF_OK;
}

int cocodiff_cache_schedule(int step, int total_steps, int warmup, int sync_interval, int *full_exchange,
                            double *r) {
    if (!full_exchange || !r || total_steps < 1 || step < 0 || step >= total_steps || warmup < 0 ||
        sync_interval < 0)
        return COCODIFF_INVALID_ARG;
    const bool refresh = sync_interval > 0 && step % sync_interval == 0;
    const bool full = step < warmup || refresh;
    const int span = total_steps - 1 - warmup;
    *full_exchange = full ? 1 : 0;
    *r = (full || span <= 0) ? 0.0 : (double)(step - warmup) / (double)span;
    return COCODIFF_OK;
}

int cocodiff_layer_step(int step, int total_steps, int warmup, int sync_interval, const uint16_t *prev_v,
                        const uint16_t *q, const uint16_t *k, const uint16_t *v, const uint16_t *wq,
                        const uint16_t *wk, float eps, const float *cs, int P, int S, int H, int D, int T,
                        int n_groups, uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                        uint16_t *q_compact, uint16_t *k_compact, uint16_t *v_compact, uint16_t *q_cache,
                        uint16_t *k_cache, uint16_t *v_cache, void *workspace, size_t workspace_bytes,
                        cocodiff_order order, void *stream_qk, void *stream_v, int64_t *sent_elements) {
    int full = 0;
    double r = 0.0;
    int rc = cocodiff_cache_schedule(step, total_steps, warmup, sync_interval, &full, &r);
    if (rc) return rc;
    if (!q_cache || !k_cache || !v_cache) return COCODIFF_INVALID_ARG;
    if (full) {
        rc = cocodiff_prologue(q, k, v, q_cache, k_cache, v_cache, wq, wk, eps, cs, P, S, H, D, order, stream_qk,
                               stream_v);
        if (rc == COCODIFF_OK && sent_elements) *sent_elements = 3LL * S * H * D;
        return rc;
    }
    rc = cocodiff_selective_prologue(prev_v, q, k, v, wq, wk, eps, cs, P, S, H, D, T, r, n_groups, metric, mask,
                                     idx, n_active, q_compact, k_compact, v_compact, q_cache, k_cache, v_cache,
                                     workspace, workspace_bytes, order, stream_qk, stream_v);
    if (rc == COCODIFF_OK && sent_elements) {
        const int n = S / T, g = n / n_groups;
        const long long act = n - (long long)n_groups * (long long)std::floor(r * (double)g);
        *sent_elements = 3LL * act * T * H * D;
    }
    return rc;
}

int cocodiff_tapa_phase1(const uint16_t *q, const uint16_t *k, const uint16_t *v, uint16_t *q_p1,
                         uint16_t *k_p1, uint16_t *v_p1, int P, int S, int H, int D, void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    if (P % 2 != 0) return COCODIFF_BAD_SHAPE;
    const size_t E = (size_t)S * H * D, bytes = E * 2;
    const uint16_t *in[3] = {q, k, v};
    uint16_t *out[3] = {q_p1, k_p1, v_p1};
    for (int i = 0; i < 3; ++i) {
        if ((in[i] == nullptr) != (out[i] == nullptr)) return COCODIFF_INVALID_ARG;
        if (!aligned16(in[i]) || !aligned16(out[i])) return COCODIFF_MISALIGNED;
    }
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) {
            if (overlap(in[i], bytes, out[j], 2 * bytes)) return COCODIFF_ALIASING;
            if (i < j && overlap(out[i], 2 * bytes, out[j], 2 * bytes)) return COCODIFF_ALIASING;
        }
    // The holdings of ring t, p1[t], are a [S][H][D] tensor: tile t keeps its own shard and
    // receives its partner's.  On one device every shard is read once and written to both
    // rings' holdings in the same pass.
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = S;
    p.H = H;
    p.D = D;
    p.src_tok = p.dst_tok = p.dst2_tok = (long long)H * D;
    p.src_head = p.dst_head = p.dst2_head = D;
    p.map = MAP_FULL;
    p.T = 1;
    set_extents(p, (long long)E, (long long)E, 0);
    p.dst2_extent = (long long)E;
    for (int i = 2; i >= 0; --i)
        if (in[i]) p.job[p.njobs++] = MoveJob{in[i], out[i], nullptr, out[i] + E};
    if (p.njobs == 0) return COCODIFF_OK;
    p.pdl = kChainedLaunch;
    CK(launch_move(p, (cudaStream_t)stream));  // a plain move of whole tensors with two destinations
    return COCODIFF_OK;
}

int cocodiff_tapa_phase2(const uint16_t *q_p1, const uint16_t *k_p1, const uint16_t *v_p1, uint16_t *q_head,
                         uint16_t *k_head, uint16_t *v_head, int P, int S, int H, int D, void *stream) {
    int rc = check_shape(P, S, H, D);
    if (rc) return rc;
    if (P % 2 != 0) return COCODIFF_BAD_SHAPE;
    const size_t bytes = (size_t)S * H * D * 2;
    const uint16_t *in[3] = {q_p1, k_p1, v_p1};
    uint16_t *out[3] = {q_head, k_head, v_head};
    for (int i = 0; i < 3; ++i) {
        if ((in[i] == nullptr) != (out[i] == nullptr)) return COCODIFF_INVALID_ARG;
        if (!aligned16(in[i]) || !aligned16(out[i])) return COCODIFF_MISALIGNED;
    }
    for (int i = 0; i < 3; ++i)
        for (int j = 0; j < 3; ++j) {
            if (overlap(in[i], 2 * bytes, out[j], bytes)) return COCODIFF_ALIASING;
            if (i < j && overlap(out[i], bytes, out[j], bytes)) return COCODIFF_ALIASING;
        }
    TapaParams tp;
    std::memset(&tp, 0, sizeof tp);
    for (int i = 2; i >= 0; --i)
        if (in[i]) { tp.src[tp.n] = in[i]; tp.dst[tp.n] = out[i]; ++tp.n; }
    tp.S = S;
    tp.H = H;
    tp.D = D;
    tp.Hl = H / P;
    tp.heads_per_block = 8;
    tp.debug = debug_counter();
    CK(launch_tapa_phase2(tp, (cudaStream_t)stream));
    return COCODIFF_OK;
}

// ---------------------------------------------------------------------------
// Scratch that lives in the library image, for callers that cannot allocate.
// One array per GPU that loads the library, held until the process exits.
constexpr size_t kStaticScratchBytes = (size_t)COCODIFF_STATIC_MAX_UNITS * 8 + 256;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

// In host code `g_static_scratch` is only a handle for the runtime, not a device
// address; the address is looked up once per device, with that device current.
static std::mutex g_static_mutex;
static void *g_static_addr[kMaxDevices];

static int static_scratch_address(void **out) {
    int dev = 0;
    CK(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return COCODIFF_INVALID_ARG;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_addr[dev]) {
        void *ptr = nullptr;
        CK(cudaGetSymbolAddress(&ptr, g_static_scratch));
        if (!ptr || (reinterpret_cast<uintptr_t>(ptr) & 255u)) return COCODIFF_MISALIGNED;
        g_static_addr[dev] = ptr;
    }
    *out = g_static_addr[dev];
    return COCODIFF_OK;
}

int cocodiff_vmajor_select_compact_static(const uint16_t *prev_v, const uint16_t *cur_v, int P, int S, int H,
                                          int D, int T, double r, int n_groups, uint64_t *metric,
                                          uint8_t *mask, int32_t *idx, int32_t *n_active,
                                          uint16_t *v_compact, void *stream) {
    // the unit count is checked against the fixed capacity before anything else is looked at
    if (T >= 1 && S >= 0 && S / T > COCODIFF_STATIC_MAX_UNITS) return COCODIFF_WORKSPACE_TOO_SMALL;
    void *scratch = nullptr;
    int rc = static_scratch_address(&scratch);
    if (rc) return rc;
    rc = check_select(prev_v, cur_v, P, S, H, D, T, r, n_groups, metric, mask, idx, n_active, scratch,
                      kStaticScratchBytes);
    if (rc) return rc;
    const uint16_t *in[3] = {nullptr, nullptr, v_compact ? cur_v : nullptr};
    uint16_t *out[3] = {nullptr, nullptr, v_compact};
    if (v_compact) {
        rc = check_tiles(in, out, S, H, D, idx, n_active);
        if (rc) return rc;
        if (overlap(prev_v, (size_t)S * H * D * 2, v_compact, (size_t)S * H * D * 2)) return COCODIFF_ALIASING;
    }
    // every piece sum the metric pass needs is stored (not accumulated) before it is read:
    // nothing in the shared array has to be cleared
    const SelectionPlan pl = plan_selection(prev_v, cur_v, S, H, D, T, r, n_groups, metric, mask, idx, n_active, scratch);
    return enqueue_select_and_pack(pl, in, out, nullptr, nullptr, nullptr, 0.f, nullptr, active_slots(S, T, r, n_groups),
                                   S, H, D, T, (cudaStream_t)stream);
}

long long cocodiff_debug_bounds_violations(void) {
#ifdef COCODIFF_DEBUG_BOUNDS
    if (!debug_counter()) return -2;
    if (cudaDeviceSynchronize() != cudaSuccess) return -2;
    unsigned long long count = 0, zero = 0;
    if (cudaMemcpyFromSymbol(&count, g_bounds_violations, sizeof count) != cudaSuccess) return -2;
    if (cudaMemcpyToSymbol(g_bounds_violations, &zero, sizeof zero) != cudaSuccess) return -2;
    return (long long)count;
#else
    return -1;
#endif
}

long long cocodiff_debug_bounds_selftest(const uint16_t *x, uint16_t *y, int S, int H, int D, void *stream) {
#ifdef COCODIFF_DEBUG_BOUNDS
    if (!x || !y || S < 2 || H < 1 || !supported_d(D) || !aligned16(x) || !aligned16(y)) return -2;
    if (cocodiff_debug_bounds_violations() < 0) return -2;  // waits and clears the counter
    // a plain [S][H][D] -> [S][H][D] move that is told its buffers end after S/2 tokens
    MoveParams p;
    std::memset(&p, 0, sizeof p);
    p.n_slots = S;
    p.H = H;
    p.D = D;
    p.src_tok = p.dst_tok = (long long)H * D;
    p.src_head = p.dst_head = D;
    p.map = MAP_FULL;
    p.T = 1;
    set_extents(p, (long long)(S / 2) * H * D, (long long)(S / 2) * H * D, 0);
    p.job[p.njobs++] = MoveJob{x, y, nullptr};
    if (launch_move(p, (cudaStream_t)stream) != cudaSuccess) return -2;
    return cocodiff_debug_bounds_violations();
#else
    (void)x; (void)y; (void)S; (void)H; (void)D; (void)stream;
    return -1;
#endif
}

}  // extern "C"

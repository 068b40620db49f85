// Shared declarations of the CUDA side of libcocodiff (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace cocodiff {

// How an output token slot o maps to source and destination tokens.
enum TokenMap : int {
    MAP_FULL = 0,     // src token = dst token = o                      (full exchange)
    MAP_GATHER = 1,   // src token = idx[o / T] * T + o % T, dst = o    (compaction)
    MAP_SCATTER = 2,  // src token = o, dst token = idx[o / T] * T + o % T  (reconstruction)
    MAP_ACTIVE = 3    // src token = dst token = idx[o / T] * T + o % T   (direct delivery: no send buffer)
};

// Programmatic dependent launch (same-stream overlap of consecutive kernels).
// A kernel launched with the programmatic attribute may start while its
// predecessor in the stream is still running; it then orders itself with
// griddepcontrol.wait, which returns once the predecessor has completed and its
// writes are visible.  Without the launch attribute these instructions do nothing.
enum PdlFlags : int {
    PDL_WAIT_AT_START = 1,   // the kernel consumes its predecessor's results
    PDL_TRIGGER = 2,         // let the successor start as soon as every block of this grid runs
    PDL_WAIT_AT_END = 4,     // independent of the predecessor, but must not complete before it
    PDL_LAUNCH_ATTR = 8      // host side: launch with programmatic stream serialization
};

// Bounds-checked build (-DCOCODIFF_DEBUG_BOUNDS): every global access of the
// kernels is checked against the extent of the buffer it belongs to; a
// violation is counted in *debug and the access is skipped (nothing traps).
// In the normal build the check is the constant `true` and costs nothing.
#ifdef COCODIFF_DEBUG_BOUNDS
#define COCODIFF_IN_BOUNDS(cond, counter) ((cond) ? true : (atomicAdd((counter), 1ull), false))
#else
#define COCODIFF_IN_BOUNDS(cond, counter) (true)
#endif

struct MoveJob {
    const uint16_t *src;
    uint16_t *dst;
    const uint16_t *w;   // RMSNorm weight [D]; nullptr = plain move
    uint16_t *dst2;      // a second destination of the same row, or nullptr: its slot of the cached
                         // head-parallel tensor [H][S][D] (gather and scatter in one pass), or the
                         // second ring's copy in phase 1 of the two-phase exchange
};

// One launch moves up to three tensors (jobs) of identical geometry.  Strides
// are in elements.  A stride given as COMPACT_STRIDE is n_active * T * D, read
// on the device.
constexpr long long COMPACT_STRIDE = -1;

struct MoveParams {
    MoveJob job[3];
    int njobs;
    int n_slots;            // token slots covered by the grid (capacity)
    int slots_exact;        // n_slots IS n_active * T (the host derived it from the rule): n_active is not read
    int H, D;
    long long src_tok, src_head, dst_tok, dst_head;
    long long dst2_tok, dst2_head;  // strides of job.dst2
    const float *cs;        // [S][D/2][2] or nullptr
    float eps;
    const int32_t *idx;     // active units (MAP_GATHER / MAP_SCATTER)
    const int32_t *n_active;
    int T;
    int n_units;            // S / T: indices read from idx are clamped to [0, n_units)
    int map;
    int pdl;                // programmatic dependent launch: see PdlFlags
    int head_split;         // blocks per tile along the heads (>= 1); set by the launcher
    long long src_extent, dst_extent;  // elements reachable from job.src / job.dst (bounds-checked build)
    long long dst2_extent;             // elements reachable from job.dst2
    long long cs_extent;               // floats reachable from cs
    unsigned long long *debug;         // violation counter (bounds-checked build), else nullptr
};

// Selection over n units in n_groups contiguous groups of g.  The metric of unit
// e is metric[e] when parts == 0, else the sum of partial[e * parts + k], k < parts
// (the pieces the metric kernel wrote); in that case the sums are also written
// to metric_out.
struct SelectParams {
    const unsigned long long *metric;   // [n], parts == 0
    const unsigned long long *partial;  // [n * parts], parts >= 1
    unsigned long long *metric_out;     // [n], parts >= 1
    int parts;
    int n, n_groups, g, n_cached;
    uint8_t *mask;
    int32_t *idx;
    int32_t *n_active;
    unsigned long long *debug;
};

// Metric pass: every unit is cut into `parts` contiguous pieces of part_vecs
// 16-byte vectors; piece (u, k) is summed by one block (warp_mode == 0) or the
// whole unit by one warp (warp_mode == 1, parts == 1) and stored, without
// atomics, to out[u * parts + k].
struct MetricParams {
    const uint4 *prev, *cur;
    unsigned long long *out;
    long long unit_vecs;          // 16-byte vectors per selection unit
    long long part_vecs;
    int parts;
    int n_units;
    int warp_mode;
    int pdl;                      // PDL_TRIGGER: dependents may start once every block streams
    unsigned long long *debug;
};

// Phase 2 of the two-phase exchange: up to three tensors, src = [2][S][H][D] (the
// copies held by ring 0 and ring 1), dst = [H][S][D].
struct TapaParams {
    const uint16_t *src[3];
    uint16_t *dst[3];
    int n;                 // tensors
    int S, H, D, Hl;       // Hl = H / P heads per rank
    int heads_per_block;
    unsigned long long *debug;
};

// How the metric pass cuts the units (host side; also sizes the workspace).
struct MetricPlan {
    int parts;
    long long part_vecs;
    int warp_mode;
};
MetricPlan plan_metric(int n_units, long long unit_vecs);

// Units up to this count are selected by every block of the consuming kernel
// itself (no selection launch); it is also the largest group the counting
// selection kernel takes.
constexpr int kCountMax = 256;

cudaError_t launch_tapa_phase2(const TapaParams &p, cudaStream_t stream);
cudaError_t launch_move(const MoveParams &p, cudaStream_t stream);
// Compaction (and scatter into job.dst2) of the active units.  sel != nullptr:
// every block first runs the selection over sel->n <= kCountMax units itself
// and block 0 publishes metric, mask, idx and n_active; sel == nullptr: the list
// is read from p.idx / p.n_active.
cudaError_t launch_selective_move(const MoveParams &p, const SelectParams *sel, cudaStream_t stream);
cudaError_t launch_rope_table(float *cs, const int32_t *pos, int S, int D, double theta, cudaStream_t stream);
// pdl: PDL_LAUNCH_ATTR | PDL_WAIT_AT_START when the metric was produced by the preceding
// kernel of the stream; PDL_TRIGGER lets the kernel after the selection start early.
cudaError_t launch_select(const SelectParams &p, cudaStream_t stream, int pdl = 0);
cudaError_t launch_metric(const MetricParams &p, cudaStream_t stream);

}  // namespace cocodiff

/*
 * libcocodiff - the per-layer Ulysses attention prologue of CoCoDiff on one
 * NVIDIA B200 (sm_100a): QK RMSNorm + 2-D RoPE, the sequence-parallel ->
 * head-parallel exchange issued V-first, and V-Major selection / compaction /
 * reconstruction.  The P ranks are virtual shards of one device's memory, so
 * the all-to-all is a device-local permutation.
 *
 * Conventions for every entry point
 *   - Returns 0 (COCODIFF_OK) or a negative cocodiff_status.  Arguments are
 *     checked before anything is enqueued: after every status except
 *     COCODIFF_CUDA_ERROR nothing has been enqueued.  COCODIFF_CUDA_ERROR means
 *     the runtime refused a launch or a copy; work that the same call enqueued
 *     before that stays enqueued, and a call that uses two streams still
 *     orders stream_qk behind stream_v before it returns.
 *   - Unless a parameter says "host", every pointer is a DEVICE pointer owned
 *     by the caller.  The library allocates no device memory, never
 *     synchronises the device and enqueues only on the streams it is given
 *     (void* = cudaStream_t, NULL = the default stream).  Calls return as soon
 *     as the work is enqueued.
 *   - Stream order holds between calls and towards the caller's own work.  On
 *     one stream the first kernel of a call is launched with programmatic
 *     stream serialization and waits (griddepcontrol.wait) for whatever
 *     precedes it before it touches memory, and the last kernel of a call lets
 *     its successor become resident while it drains, so consecutive calls
 *     overlap launch latency, ramp-up and drain.  A kernel of the caller that
 *     follows a call is not affected unless the caller launches it with the
 *     same attribute; it then has to call cudaGridDependencySynchronize()
 *     before it reads the call's outputs, as the programming model requires.
 *   - bf16 tensors are passed as uint16_t bit patterns, row-major, last index
 *     fastest, and must be 16-byte aligned.  Head dimension D is a multiple of
 *     8 from 8 to 256 (a row is D/8 16-byte vectors, one per lane of a group of
 *     lanes; powers of two use every lane of the group).
 *   - Layouts:  SEQ  = [P][S/P][H][D] == [S][H][D]  (rank p owns tokens
 *                      [p*S/P, (p+1)*S/P): the sequence-parallel layout)
 *               HEAD = [P][H/P][S][D] == [H][S][D]  (rank p owns heads
 *                      [p*H/P, (p+1)*H/P): the head-parallel layout)
 *     (Section II-A of the paper.)  P must divide S and H, and P <= H: one
 *     head per rank is the Ulysses limit (Section IV-B).
 *   - A selection unit is T consecutive tokens of one source rank, all heads
 *     (T = 1 is the paper's per-token rule); T must divide S/P.
 *     COMPACT = [H][n_active][T][D] == [P][H/P][n_active*T][D]: what each
 *     destination rank receives when only the active units are sent, source
 *     ranks concatenated in rank order (ascending unit index).
 */
#ifndef COCODIFF_H
#define COCODIFF_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    COCODIFF_OK = 0,
    COCODIFF_INVALID_ARG = -1,         /* null pointer, P < 1, r outside [0,1], bad enum          */
    COCODIFF_BAD_SHAPE = -2,           /* P does not divide S or H, P > H, unsupported D, T, groups */
    COCODIFF_MISALIGNED = -3,          /* a tensor pointer is not 16-byte aligned                  */
    COCODIFF_WORKSPACE_TOO_SMALL = -4,
    COCODIFF_CUDA_ERROR = -5,          /* a launch or copy failed; see cocodiff_last_cuda_error()  */
    COCODIFF_ALIASING = -6             /* input and output overlap where that is not allowed       */
} cocodiff_status;

/* Order of issue of the three exchanges (Section III-C, "V-First Scheduling").
 * LUMP: Q, K and V leave together in one launch on stream_qk (the flat order).
 * V_FIRST: V's exchange is launched first.  With two streams it runs on stream_v
 * beside the norm + RoPE + exchange of Q and K on stream_qk.  With stream_v ==
 * stream_qk the two launches share the stream and are chained with a programmatic
 * dependent launch: Q/K's grid starts while V's last blocks drain and completes
 * after it.  Results are identical in every case. */
typedef enum { COCODIFF_LUMP = 0, COCODIFF_V_FIRST = 1 } cocodiff_order;

const char *cocodiff_status_string(int status);
int cocodiff_version(void);
/* cudaError_t of the most recent COCODIFF_CUDA_ERROR on the calling thread (0 if none). */
int cocodiff_last_cuda_error(void);

/* RoPE angle table (Section II-B, "Rotary position embeddings"; axial 2-D form).
 * cs[s][p] = (cos, sin) of pos[s][axis] * theta^(-2i/(D/2)) with axis = p / (D/4),
 * i = p % (D/4): the first D/4 pairs (dimensions [0, D/2)) rotate with the row
 * position, the last D/4 with the column position.  cs: [S][D/2][2] float out;
 * pos: [S][2] int32 (row, col).  Evaluated in double on the device, rounded to
 * float.  Built once per resolution, not per layer. */
int cocodiff_rope_table_2d(float *cs, const int32_t *pos, int S, int D, double theta, void *stream);

/* QK normalisation + RoPE alone (Section II-B), SEQ in -> SEQ out.
 * y = RoPE(x * rsqrt(mean_D(x^2) + eps) * w), per (token, head), fp32 arithmetic,
 * one round-to-nearest-even to bf16.  Pair (2p, 2p+1) is rotated by cs[s][p].
 * Inputs are expected finite with squares representable in fp32 (|x| < 1.8e19);
 * NaN, Inf and eps = 0 with an all-zero row give unspecified bit patterns.
 * q/k may be NULL to skip that tensor; out == in (same tensor) is allowed,
 * any other overlap is COCODIFF_ALIASING.  wq, wk: [D] bf16.  cs may be NULL
 * (no rotation). */
int cocodiff_qk_norm_rope(const uint16_t *q, const uint16_t *k, uint16_t *q_out, uint16_t *k_out,
                          const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                          int S, int H, int D, void *stream);

/* The Ulysses exchange alone (Section II-A): SEQ -> HEAD, bit-exact move.
 * Any of the (x, x_head) pairs may be NULL/NULL to skip it.  With V_FIRST and
 * stream_v != stream_qk, stream_v first waits for the work already enqueued
 * on stream_qk, and stream_qk afterwards waits for V: to the caller the call
 * is ordered on stream_qk. */
int cocodiff_ulysses_a2a(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                         uint16_t *q_head, uint16_t *k_head, uint16_t *v_head,
                         int P, int S, int H, int D, cocodiff_order order,
                         void *stream_qk, void *stream_v);

/* The second all-to-all of Section II-A: HEAD -> SEQ, bit-exact move. */
int cocodiff_ulysses_a2a_inverse(const uint16_t *q_head, const uint16_t *k_head, const uint16_t *v_head,
                                 uint16_t *q, uint16_t *k, uint16_t *v,
                                 int P, int S, int H, int D, void *stream);

/* The fused prologue of one layer, full exchange (Sections II-B, II-A, III-C):
 * every (token, head) row of Q and K is read once, normalised, rotated and
 * written straight into its HEAD slot; V is moved untouched, first.  Stream
 * semantics as for cocodiff_ulysses_a2a.  A (x, x_head) pair may be NULL/NULL to
 * leave that tensor out (a layer normally passes all three). */
int cocodiff_prologue(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      uint16_t *q_head, uint16_t *k_head, uint16_t *v_head,
                      const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                      int P, int S, int H, int D, cocodiff_order order,
                      void *stream_qk, void *stream_v);

/* The same prologue for HOST tensors: q, k, v and the three results are host
 * pointers (pinned memory makes the copies asynchronous); dev_in and dev_out
 * are caller-owned device staging buffers of 3*S*H*D bf16 each.  With V_FIRST
 * and two streams the tokens are processed in chunks that alternate between
 * the streams, so that host-to-device copies, the kernel and device-to-host
 * copies of neighbouring chunks overlap; inside a chunk V leads.  With LUMP (or
 * equal streams) everything runs in order on stream_qk.  wq, wk, cs stay device
 * pointers.  On return stream_qk is ordered after all of it. */
int cocodiff_prologue_host(const uint16_t *q_host, const uint16_t *k_host, const uint16_t *v_host,
                           uint16_t *q_head_host, uint16_t *k_head_host, uint16_t *v_head_host,
                           uint16_t *dev_in, uint16_t *dev_out,
                           const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                           int P, int S, int H, int D, cocodiff_order order,
                           void *stream_qk, void *stream_v);

/* V-Major active-projection selection (Section III-D, "Active projection
 * selection") and compaction of V.
 *   metric[u] = sum over the unit's T*H*D elements of fix(|cur - prev|), where
 *     the difference is one fp32 subtraction and fix(d) = min(trunc(d * 2^16),
 *     2^32 - 1) (NaN -> 2^32 - 1): an integer L1 distance, independent of the
 *     order of accumulation.
 *   The n = S/T units form n_groups contiguous groups of g units (1 = one
 *     global decision, P/2 = the paper's per-GPU scope, P = per rank).  In each
 *     group the floor(r * g) units smallest by (metric, index) are cached
 *     (mask 0), the others active (mask 1).
 *   idx[0 .. n_active) = the active units, ascending; n_active is written to
 *     device memory (the host can compute it: n - n_groups * floor(r * g)).
 *   v_compact, if not NULL: COMPACT layout of the active units of cur_v
 *     (capacity S*H*D elements).
 * prev_v is only read: which step it holds is the caller's policy.
 * workspace: cocodiff_vmajor_workspace_bytes() bytes of scratch, 256-byte
 * aligned; contents are undefined on entry and on exit.  Large units are cut
 * into pieces that are summed by different thread blocks; the workspace holds
 * one 64-bit sum per piece (each is stored before it is read, so nothing has
 * to be cleared).  Concurrent calls need distinct workspaces. */
size_t cocodiff_vmajor_workspace_bytes(int P, int S, int H, int D, int T);
int cocodiff_vmajor_select_compact(const uint16_t *prev_v, const uint16_t *cur_v,
                                   int P, int S, int H, int D, int T, double r, int n_groups,
                                   uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                                   uint16_t *v_compact,
                                   void *workspace, size_t workspace_bytes, void *stream);

/* Selection alone from a given metric array (the rule of the same passage);
 * used by the call above and exposed for tests and for callers that keep their
 * own metric. */
int cocodiff_vmajor_select(const uint64_t *metric, int n, double r, int n_groups,
                           uint8_t *mask, int32_t *idx, int32_t *n_active, void *stream);

/* Extraction of the active units of one tensor into COMPACT (Section III-D,
 * "Selective communication in TAPA").  w != NULL: the rows are normalised and
 * rotated on the way (Q, K); w == NULL: plain move (V).  idx and n_active are
 * read on the device, so no host round trip separates selection and packing.
 * x_compact capacity: S*H*D elements. */
int cocodiff_pack_active(const uint16_t *x, const uint16_t *w, float eps, const float *cs,
                         const int32_t *idx, const int32_t *n_active, uint16_t *x_compact,
                         int P, int S, int H, int D, int T, void *stream);

/* The same extraction for Q, K and V in one launch (Q, K normalised and rotated,
 * V moved); any (x, x_compact) pair may be NULL/NULL. */
int cocodiff_pack_active_qkv(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                             const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                             const int32_t *idx, const int32_t *n_active,
                             uint16_t *q_compact, uint16_t *k_compact, uint16_t *v_compact,
                             int P, int S, int H, int D, int T, void *stream);

/* Receiver-side reconstruction (Section III-D, "Post-Phase 2"): indexed scatter
 * x_cache[h][idx[a]*T + j][:] = x_compact[h][a][j][:]; all other rows of the
 * cached HEAD tensor keep their bits. */
int cocodiff_unpack(const uint16_t *x_compact, const int32_t *idx, const int32_t *n_active,
                    uint16_t *x_cache, int P, int S, int H, int D, int T, void *stream);

/* The same scatter for Q, K and V in one launch; any pair may be NULL/NULL. */
int cocodiff_unpack_qkv(const uint16_t *q_compact, const uint16_t *k_compact, const uint16_t *v_compact,
                        const int32_t *idx, const int32_t *n_active,
                        uint16_t *q_cache, uint16_t *k_cache, uint16_t *v_cache,
                        int P, int S, int H, int D, int T, void *stream);

/* One selective step of a layer (Section III-D; timeline of Figure 4(d)):
 * metric and selection on V, compaction of the active units of V (moved) and of
 * Q, K (normalised and rotated on the way), then - if the three caches are
 * given - the scatter over the cached HEAD tensors.  V_FIRST with two streams:
 * metric, selection and V's compaction run on stream_v, Q and K follow on
 * stream_qk when V's part is done; LUMP or equal streams: one stream, the three
 * compactions in one launch.  Consecutive kernels of a stream are chained with
 * programmatic dependent launches.  Stream semantics as for
 * cocodiff_ulysses_a2a; outputs and workspace as for
 * cocodiff_vmajor_select_compact.  The caches are all given or all NULL.
 * Direct delivery: with the caches given, the three compact buffers may all be
 * NULL; the active rows are then stored straight to their slots of the cached
 * HEAD tensors (between NVLink peers: a store into the receiver's memory) and
 * no send buffer is written.  The caches end up with the same bits either way.
 * Compact buffers that are given are all given; all NULL without the caches is
 * INVALID_ARG. */
int cocodiff_selective_prologue(const uint16_t *prev_v, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                                const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                                int P, int S, int H, int D, int T, double r, int n_groups,
                                uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                                uint16_t *q_compact, uint16_t *k_compact, uint16_t *v_compact,
                                uint16_t *q_cache, uint16_t *k_cache, uint16_t *v_cache,
                                void *workspace, size_t workspace_bytes, cocodiff_order order,
                                void *stream_qk, void *stream_v);

/* Time-varying cache schedule (Section III-D, "Time-varying cache scheduling"),
 * host-only arithmetic, steps numbered from 0:
 *   - the first `warmup` steps and every step with step % sync_interval == 0
 *     (sync_interval > 0) are full exchanges: *full_exchange = 1, *r = 0;
 *   - otherwise *full_exchange = 0 and the cache ratio grows linearly from 0 at
 *     step `warmup` to 1 at the last step: *r = (step - warmup) / (total_steps - 1 - warmup).
 * The paper's experiments use total_steps = 50, warmup = 5, sync_interval = 10.
 * full_exchange and r are HOST pointers. */
int cocodiff_cache_schedule(int step, int total_steps, int warmup, int sync_interval,
                            int *full_exchange, double *r);

/* One denoising step of one layer under that schedule: a full step runs
 * cocodiff_prologue straight into the three caches (resetting them to the exact
 * values of this step); a selective step runs cocodiff_selective_prologue with
 * the scheduled r.  All arguments as in those two calls; the caches are
 * required, the compact buffers may all be NULL (direct delivery).  sent_elements (HOST pointer, may be NULL) receives the number of
 * bf16 elements of Q, K, V that cross the exchange in this step. */
int cocodiff_layer_step(int step, int total_steps, int warmup, int sync_interval,
                        const uint16_t *prev_v, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                        const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                        int P, int S, int H, int D, int T, int n_groups,
                        uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                        uint16_t *q_compact, uint16_t *k_compact, uint16_t *v_compact,
                        uint16_t *q_cache, uint16_t *k_cache, uint16_t *v_cache,
                        void *workspace, size_t workspace_bytes, cocodiff_order order,
                        void *stream_qk, void *stream_v, int64_t *sent_elements);

/* Tile-aware parallel all-to-all on virtual ranks (Section III-B, TAPA): ranks 2g
 * and 2g+1 are the two tiles of GPU g; P must be even.  The two phases compose to
 * cocodiff_ulysses_a2a bit for bit; they exist to reproduce the paper's data flow
 * (what each tile holds after Phase 1, which the per-GPU selection scope works
 * on), not to be faster: inside one device - and inside one NVLink domain -
 * there is no bandwidth hierarchy to align to.
 *
 * Phase 1 (intra-GPU): the two tiles of a GPU swap their whole shards, so each
 * tile holds all tokens of its GPU.  x_p1 = [2][P/2][2*S/P][H][D], x_p1[t][g] =
 * holdings of tile t of GPU g (2*S*H*D elements per tensor); x_p1[t] as a whole
 * is a [S][H][D] tensor, so V's x_p1[0] can be given directly to the V-Major
 * calls (n_groups = P/2 is the per-GPU scope of the paper).  On one device a
 * shard is read once and written to both rings' holdings in the same pass.
 * Phase 2 (inter-GPU): one all-to-all per ring t (tile t of every GPU), no
 * traffic between rings: rank 2*g2+t takes its heads from x_p1[t] only.
 * Any (in, out) pair may be NULL/NULL. */
int cocodiff_tapa_phase1(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                         uint16_t *q_p1, uint16_t *k_p1, uint16_t *v_p1,
                         int P, int S, int H, int D, void *stream);
int cocodiff_tapa_phase2(const uint16_t *q_p1, const uint16_t *k_p1, const uint16_t *v_p1,
                         uint16_t *q_head, uint16_t *k_head, uint16_t *v_head,
                         int P, int S, int H, int D, void *stream);

/* cocodiff_vmajor_select_compact for callers that cannot allocate device memory.
 * (The paper has no counterpart: this is a deployment convenience of this library.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits - a plug-in inside
 * a serving process whose memory pool is owned by someone else, a hook that runs
 * while the application is in a no-allocation phase, a real-time loop that must
 * not touch the allocator.  Such callers already own their inputs and outputs
 * but have nowhere to get the small scratch area the metric pass needs (the
 * 64-bit sums of the pieces that large units are cut into).  Here that scratch is
 * a fixed array inside the library image on the device: COCODIFF_STATIC_MAX_UNITS
 * 64-bit words plus 256 bytes (about 256 KB), present on every GPU that
 * loads the library until the process exits.
 *
 * Arguments and results are exactly those of cocodiff_vmajor_select_compact
 * without `workspace` / `workspace_bytes`.  Differences to know about:
 *   - S / T may not exceed COCODIFF_STATIC_MAX_UNITS; more units are refused
 *     with COCODIFF_WORKSPACE_TOO_SMALL and nothing is enqueued.
 *   - The first call on each device looks up the array's device address (with
 *     that device current) and remembers it.  Make that first call outside any
 *     stream capture.
 *   - Every call on a device shares the one array, which still holds whatever
 *     the previous call left; nothing in it has to start at zero, because a
 *     call stores every word it is going to read before it reads it.  Two calls
 *     whose work overlaps on the GPU (different streams, no ordering between
 *     them) race on the array and give wrong selections: order them, or use the
 *     workspace-taking call.
 *   - No cudaMalloc, cudaFree or other allocating routine is called. */
#define COCODIFF_STATIC_MAX_UNITS 32768
int cocodiff_vmajor_select_compact_static(const uint16_t *prev_v, const uint16_t *cur_v,
                                          int P, int S, int H, int D, int T, double r, int n_groups,
                                          uint64_t *metric, uint8_t *mask, int32_t *idx, int32_t *n_active,
                                          uint16_t *v_compact, void *stream);

/* Diagnostic for the bounds-checked build of this library (compiled with
 * -DCOCODIFF_DEBUG_BOUNDS; build.py --debug-bounds writes libcocodiff_debug.so).
 * (The paper has no counterpart.)  In that build every global access of every
 * kernel is checked against the extent of the buffer it belongs to; an access
 * outside is counted and skipped, never performed and never trapped.  This
 * call waits for the device, returns the number of such accesses on the current
 * device since the previous call and resets the counter; -2 on a CUDA error.
 * The normal build carries no checks: there the call returns -1. */
long long cocodiff_debug_bounds_violations(void);

/* Self-test of that checker (bounds-checked build only; -1 in the normal build,
 * -2 on bad arguments or a CUDA error): moves x [S][H][D] to y while claiming
 * that both buffers end after S/2 tokens.  The accesses beyond are in fact
 * inside the caller's buffers, so nothing is harmed; the checker must count
 * and skip each of them.  Returns the count: 2 * (S - S/2) * H * D/8 (one load
 * and one store per 16-byte vector); y keeps its old contents beyond S/2. */
long long cocodiff_debug_bounds_selftest(const uint16_t *x, uint16_t *y, int S, int H, int D, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* COCODIFF_H */

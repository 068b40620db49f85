/*
 * CPU oracle for the Ulysses attention-prologue path of CoCoDiff.
 *
 * TEST INFRASTRUCTURE ONLY.  Plain, slow C; it shares no code with the CUDA
 * library and the product never calls it.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may load this file.  The normal build is
 * single-threaded.  The benchmark also builds the same source with -fopenmp to
 * time it on all host cores: the `omp` pragmas below then spread independent
 * outer loops (tokens, messages, units) over the threads; without that flag they
 * are ignored, and they change no arithmetic either way.
 *
 * What is written out here, with the passage of the paper each part follows:
 *   - the sequence-parallel -> head-parallel exchange of Ulysses (Section II-A)
 *     as an explicit (source rank, destination rank) message loop, and its
 *     inverse (the second all-to-all of the same section);
 *   - QK normalisation (RMSNorm) and rotary embeddings on Q and K, never on V
 *     (Section II-B, "QK normalization" and "Rotary position embeddings");
 *   - the two phases of the tile-aware parallel all-to-all (Section III-B);
 *   - the V-Major rule (Section III-D, "Active projection selection"): an L1
 *     distance between the current and the cached value vectors, the fraction
 *     r with the smallest distances is cached, the rest is active;
 *   - extraction of the active projections before the exchange (Section III-D,
 *     "Selective communication in TAPA") and the receiver-side indexed scatter
 *     over the cached head-parallel tensors ("Post-Phase 2").
 *
 * Readings taken where the paper gives no formula:
 *   - RMSNorm is per (token, head) over the D head dimensions, eps inside the
 *     square root, one bf16 weight vector [D] per tensor.
 *   - RoPE is axial 2-D: the first D/2 dimensions rotate with the row position,
 *     the last D/2 with the column position; adjacent elements (2p, 2p+1) form
 *     a pair; frequency i of an axis is theta^(-2i/(D/2)), i in [0, D/4).
 *   - storage is bf16, arithmetic is fp32 with one round-to-nearest-even at the
 *     end; the sum of squares and the transcendental functions are evaluated
 *     in double and rounded to fp32 (this side is the accurate one).
 *   - the L1 distance is accumulated as an integer: each |cur - prev| (one
 *     fp32 subtraction) is scaled by 2^16, truncated and saturated to 32 bits,
 *     NaN counts as the saturated value; the sum is 64-bit.  The sum is then
 *     independent of the order of accumulation, so a mask can be exact.
 *   - a selection unit is T consecutive tokens (all heads); T = 1 is the
 *     paper's per-token rule.  Units are ordered by (distance, index); in each
 *     of n_groups contiguous groups of g units the first floor(r*g) are cached.
 *
 * Parity pins (tests/test_oracle_*.py, none of them re-types these formulas):
 * exchange - closed form HEAD[h][s] = SEQ[s][h] for every P, bijection, index
 * fill, sizes printed in the paper; TAPA - each tile holds its GPU's tokens, the
 * two phases compose to the flat exchange, rings are independent; norm - unit RMS, power-of-two scale
 * invariance, 3-4-5 hand case, fp64 textbook evaluation; RoPE - identity at
 * position 0, pair-norm preservation, relative-position property, quarter
 * turn, axis separation, complex-multiplication form; metric - brute force,
 * single-element change; selection - sort-based reference with ties, r = 0 and
 * r = 1; compaction/unpack - elementwise definition.  Unpinned: agreement with
 * the paper's own implementation (pairing convention, eps, tie-break), whose
 * code is not available; "parity unpinned" applies to that only.
 *
 * Layouts (bf16 bit patterns as uint16_t, row-major, last index fastest):
 *   SEQ  = [P][S/P][H][D]  ==  [S][H][D]   rank p owns tokens [p*S/P, (p+1)*S/P)
 *   HEAD = [P][H/P][S][D]  ==  [H][S][D]   rank p owns heads  [p*H/P, (p+1)*H/P)
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_BAD (-1)

static float bf16_to_f32(uint16_t b) {
    uint32_t u = (uint32_t)b << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return f;
}

/* round to nearest, ties to even */
static uint16_t f32_to_bf16(float f) {
    uint32_t u;
    memcpy(&u, &f, sizeof u);
    if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x0040u);
    u += 0x7fffu + ((u >> 16) & 1u);
    return (uint16_t)(u >> 16);
}

int oracle_version(void) { return 1; }

/* exposed so that tests can pin the conversion against exhaustive checks */
float oracle_bf16_to_f32(uint16_t b) { return bf16_to_f32(b); }
uint16_t oracle_f32_to_bf16(float f) { return f32_to_bf16(f); }

/* Number of elements of one tensor that a rank holds after the exchange: all S
 * tokens of H/P heads (Section II-A; the same count underlies the per-tile
 * cache size of Section III-D, "Memory overhead analysis"). */
int64_t oracle_head_shard_elems(int P, int S, int H, int D) {
    return (int64_t)(H / P) * S * D;
}

/* Elements one rank sends per tensor: its S/P tokens, all heads (the per-rank
 * message of the running example in Section III-B). */
int64_t oracle_seq_shard_elems(int P, int S, int H, int D) {
    return (int64_t)(S / P) * H * D;
}

/* ------------------------------------------------------------------------ */
/* RoPE angle table: cs[s][p] = (cos, sin) of pos[s][axis(p)] * freq(p).    */
/* Section II-B, "Rotary position embeddings"; axial 2-D reading.           */
int oracle_rope_table_2d(float *cs, const int32_t *pos, int S, int D, double theta) {
    if (D % 4 != 0) return ORACLE_BAD;
    const int n = D / 4; /* pairs per axis */
    for (int s = 0; s < S; ++s) {
        for (int p = 0; p < D / 2; ++p) {
            const int axis = p / n;
            const int i = p % n;
            const double freq = pow(theta, -2.0 * (double)i / (double)(D / 2));
            const double phi = (double)pos[2 * s + axis] * freq;
            cs[((size_t)s * (D / 2) + p) * 2 + 0] = (float)cos(phi);
            cs[((size_t)s * (D / 2) + p) * 2 + 1] = (float)sin(phi);
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* RMSNorm then RoPE on one tensor in SEQ layout (Section II-B).            */
/* y_f32 (optional) receives the fp32 values before the final rounding,     */
/* y_bf16 (optional) the rounded result.  cs == NULL skips the rotation,    */
/* w == NULL skips the normalisation.                                       */
int oracle_norm_rope(const uint16_t *x, const uint16_t *w, float eps, const float *cs,
                     int S, int H, int D, uint16_t *y_bf16, float *y_f32) {
    if (D % 2 != 0 || D < 2 || D > 65536) return ORACLE_BAD;
#pragma omp parallel for schedule(static)
    for (int s = 0; s < S; ++s) {
        float row[D]; /* one row at a time, private to the token's loop iteration */
        for (int h = 0; h < H; ++h) {
            const size_t base = ((size_t)s * H + h) * D;
            for (int j = 0; j < D; ++j) row[j] = bf16_to_f32(x[base + j]);
            if (w) {
                double acc = 0.0;
                for (int j = 0; j < D; ++j) acc += (double)row[j] * (double)row[j];
                const float ms = (float)(acc / (double)D);
                const float inv = (float)(1.0 / sqrt((double)ms + (double)eps));
                for (int j = 0; j < D; ++j) {
                    const float t = row[j] * inv;
                    row[j] = t * bf16_to_f32(w[j]);
                }
            }
            if (cs) {
                for (int p = 0; p < D / 2; ++p) {
                    const float c = cs[((size_t)s * (D / 2) + p) * 2 + 0];
                    const float sn = cs[((size_t)s * (D / 2) + p) * 2 + 1];
                    const float a = row[2 * p], b = row[2 * p + 1];
                    const float ac = a * c, bs = b * sn, as = a * sn, bc = b * c;
                    row[2 * p] = ac - bs;
                    row[2 * p + 1] = as + bc;
                }
            }
            for (int j = 0; j < D; ++j) {
                if (y_f32) y_f32[base + j] = row[j];
                if (y_bf16) y_bf16[base + j] = f32_to_bf16(row[j]);
            }
        }
    }
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Ulysses exchange, SEQ -> HEAD (Section II-A): every source rank cuts its  */
/* tokens into P messages by destination head range, the messages cross,    */
/* every destination lays the P received messages out by source token range. */
static int shapes_ok(int P, int S, int H, int D) {
    return P >= 1 && S >= 0 && H >= 1 && D >= 1 && S % P == 0 && H % P == 0;
}

int oracle_ulysses_a2a(const uint16_t *seq, uint16_t *head, int P, int S, int H, int D) {
    if (!shapes_ok(P, S, H, D)) return ORACLE_BAD;
    const int Sl = S / P, Hl = H / P;
    const size_t msg = (size_t)Sl * Hl * D; /* elements per (src, dst) message */
    const size_t E = (size_t)S * H * D;
    uint16_t *sendbuf = (uint16_t *)malloc(2 * (E ? E : 1));
    uint16_t *recvbuf = (uint16_t *)malloc(2 * (E ? E : 1));
    if (!sendbuf || !recvbuf) { free(sendbuf); free(recvbuf); return ORACLE_BAD; }
    /* pack: sendbuf[src][dst][s_l][h_l][:] */
#pragma omp parallel for collapse(2) schedule(static)
    for (int src = 0; src < P; ++src)
        for (int dst = 0; dst < P; ++dst)
            for (int sl = 0; sl < Sl; ++sl)
                for (int hl = 0; hl < Hl; ++hl) {
                    const uint16_t *from = seq + (((size_t)src * Sl + sl) * H + (size_t)dst * Hl + hl) * D;
                    uint16_t *to = sendbuf + ((size_t)src * P + dst) * msg + ((size_t)sl * Hl + hl) * D;
                    memcpy(to, from, 2 * (size_t)D);
                }
    /* the wire: recvbuf[dst][src] = sendbuf[src][dst] */
#pragma omp parallel for collapse(2) schedule(static)
    for (int src = 0; src < P; ++src)
        for (int dst = 0; dst < P; ++dst)
            memcpy(recvbuf + ((size_t)dst * P + src) * msg, sendbuf + ((size_t)src * P + dst) * msg, 2 * msg);
    /* unpack: HEAD[dst][h_l][src*Sl + s_l][:] */
#pragma omp parallel for collapse(2) schedule(static)
    for (int dst = 0; dst < P; ++dst)
        for (int src = 0; src < P; ++src)
            for (int sl = 0; sl < Sl; ++sl)
                for (int hl = 0; hl < Hl; ++hl) {
                    const uint16_t *from = recvbuf + ((size_t)dst * P + src) * msg + ((size_t)sl * Hl + hl) * D;
                    uint16_t *to = head + (((size_t)dst * Hl + hl) * S + (size_t)src * Sl + sl) * D;
                    memcpy(to, from, 2 * (size_t)D);
                }
    free(sendbuf);
    free(recvbuf);
    return ORACLE_OK;
}

/* The second all-to-all of Section II-A: HEAD -> SEQ.  Here rank `src` owns  */
/* heads and sends to rank `dst` the tokens that dst owns.                    */
int oracle_ulysses_a2a_inverse(const uint16_t *head, uint16_t *seq, int P, int S, int H, int D) {
    if (!shapes_ok(P, S, H, D)) return ORACLE_BAD;
    const int Sl = S / P, Hl = H / P;
    const size_t msg = (size_t)Sl * Hl * D;
    const size_t E = (size_t)S * H * D;
    uint16_t *sendbuf = (uint16_t *)malloc(2 * (E ? E : 1));
    uint16_t *recvbuf = (uint16_t *)malloc(2 * (E ? E : 1));
    if (!sendbuf || !recvbuf) { free(sendbuf); free(recvbuf); return ORACLE_BAD; }
    for (int src = 0; src < P; ++src)
        for (int dst = 0; dst < P; ++dst)
            for (int hl = 0; hl < Hl; ++hl)
                for (int sl = 0; sl < Sl; ++sl) {
                    const uint16_t *from = head + (((size_t)src * Hl + hl) * S + (size_t)dst * Sl + sl) * D;
                    uint16_t *to = sendbuf + ((size_t)src * P + dst) * msg + ((size_t)hl * Sl + sl) * D;
                    memcpy(to, from, 2 * (size_t)D);
                }
    for (int src = 0; src < P; ++src)
        for (int dst = 0; dst < P; ++dst)
            memcpy(recvbuf + ((size_t)dst * P + src) * msg, sendbuf + ((size_t)src * P + dst) * msg, 2 * msg);
    for (int dst = 0; dst < P; ++dst)
        for (int src = 0; src < P; ++src)
            for (int hl = 0; hl < Hl; ++hl)
                for (int sl = 0; sl < Sl; ++sl) {
                    const uint16_t *from = recvbuf + ((size_t)dst * P + src) * msg + ((size_t)hl * Sl + sl) * D;
                    uint16_t *to = seq + (((size_t)dst * Sl + sl) * H + (size_t)src * Hl + hl) * D;
                    memcpy(to, from, 2 * (size_t)D);
                }
    free(sendbuf);
    free(recvbuf);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Tile-aware parallel all-to-all (TAPA, Section III-B).  Ranks 2g and 2g+1    */
/* are the two tiles of GPU g; P must be even.                                 */
/* Phase 1: inside every GPU the two tiles swap their whole shards (S/P tokens,*/
/* all heads - 14 MB for Q, K, V together in the running example), so         */
/* that afterwards each tile holds all tokens of its GPU in token order.       */
/* p1 layout: [2][P/2][2*S/P][H][D], p1[t][g] = what tile t of GPU g holds.    */
/* With this layout p1[t] as a whole is again a [S][H][D] tensor.              */
int oracle_tapa_phase1(const uint16_t *seq, uint16_t *p1, int P, int S, int H, int D) {
    if (!shapes_ok(P, S, H, D) || P % 2 != 0) return ORACLE_BAD;
    const int Sl = S / P, G = P / 2;
    const size_t shard = (size_t)Sl * H * D; /* elements one tile owns and sends */
    uint16_t *message = (uint16_t *)malloc(2 * (shard ? shard : 1));
    if (!message) return ORACLE_BAD;
    for (int g = 0; g < G; ++g)
        for (int t = 0; t < 2; ++t) {
            const int me = 2 * g + t, partner = 2 * g + (1 - t);
            uint16_t *held = p1 + ((size_t)t * G + g) * 2 * shard; /* [2*Sl][H][D] */
            /* own shard stays, at the position of tile t */
            memcpy(held + (size_t)t * shard, seq + (size_t)me * shard, 2 * shard);
            /* the partner's shard arrives as one message */
            memcpy(message, seq + (size_t)partner * shard, 2 * shard);
            memcpy(held + (size_t)(1 - t) * shard, message, 2 * shard);
        }
    free(message);
    return ORACLE_OK;
}

/* Phase 2: two independent all-to-alls among the P/2 tiles of each ring      */
/* (ring t = tile t of every GPU), no traffic between the rings.  Tile (g,t)   */
/* sends to tile (g2,t) the tokens of GPU g restricted to the heads of rank    */
/* 2*g2+t; the receiver lays the messages out by source GPU.                   */
int oracle_tapa_phase2(const uint16_t *p1, uint16_t *head, int P, int S, int H, int D) {
    if (!shapes_ok(P, S, H, D) || P % 2 != 0) return ORACLE_BAD;
    const int Sl = S / P, Hl = H / P, G = P / 2, Sg = 2 * Sl; /* Sg tokens per GPU */
    const size_t msg = (size_t)Sg * Hl * D;
    uint16_t *message = (uint16_t *)malloc(2 * (msg ? msg : 1));
    if (!message) return ORACLE_BAD;
    for (int t = 0; t < 2; ++t)
        for (int g = 0; g < G; ++g)
            for (int g2 = 0; g2 < G; ++g2) {
                const uint16_t *held = p1 + ((size_t)t * G + g) * Sg * H * D;
                const int dst = 2 * g2 + t;
                for (int j = 0; j < Sg; ++j)
                    for (int hl = 0; hl < Hl; ++hl)
                        memcpy(message + ((size_t)j * Hl + hl) * D,
                               held + ((size_t)j * H + (size_t)dst * Hl + hl) * D, 2 * (size_t)D);
                for (int j = 0; j < Sg; ++j)
                    for (int hl = 0; hl < Hl; ++hl)
                        memcpy(head + (((size_t)dst * Hl + hl) * S + (size_t)g * Sg + j) * D,
                               message + ((size_t)j * Hl + hl) * D, 2 * (size_t)D);
            }
    free(message);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* V-Major metric (Section III-D, "Active projection selection"): L1 distance */
/* between the current and the cached value vectors of each selection unit.  */
/* Unit u = tokens [u*T, (u+1)*T), all heads; T must divide S/P so that a    */
/* unit never straddles two source ranks.                                    */
static uint64_t fix16(float d) {
    if (d != d) return 0xffffffffull;            /* NaN */
    const double scaled = (double)d * 65536.0;   /* exact */
    if (scaled >= 4294967295.0) return 0xffffffffull;
    return (uint64_t)scaled;                     /* truncation; d >= 0 */
}

int oracle_vmajor_metric(const uint16_t *prev_v, const uint16_t *cur_v, int P, int S, int H,
                         int D, int T, uint64_t *metric) {
    if (!shapes_ok(P, S, H, D) || T < 1 || (S / P) % T != 0) return ORACLE_BAD;
    const int n = S / T;
    const size_t unit = (size_t)T * H * D;
#pragma omp parallel for schedule(static)
    for (int u = 0; u < n; ++u) {
        uint64_t acc = 0;
        for (size_t e = 0; e < unit; ++e) {
            const float c = bf16_to_f32(cur_v[(size_t)u * unit + e]);
            const float p = bf16_to_f32(prev_v[(size_t)u * unit + e]);
            const float diff = c - p;
            acc += fix16(fabsf(diff));
        }
        metric[u] = acc;
    }
    return ORACLE_OK;
}

/* Selection (same passage): in each group the floor(r*g) units with the     */
/* smallest (metric, index) are cached (mask 0); the others are active       */
/* (mask 1).  idx lists the active units ascending - the small integer list  */
/* that the paper all-gathers; on one device the gather is a concatenation.  */
typedef struct { uint64_t m; int32_t i; } keyed;

static int keyed_cmp(const void *a, const void *b) {
    const keyed *x = (const keyed *)a, *y = (const keyed *)b;
    if (x->m != y->m) return x->m < y->m ? -1 : 1;
    if (x->i != y->i) return x->i < y->i ? -1 : 1;
    return 0;
}

int oracle_vmajor_select(const uint64_t *metric, int n, int n_groups, double r,
                         uint8_t *mask, int32_t *idx, int32_t *n_active) {
    if (n < 0 || n_groups < 1 || n % n_groups != 0 || !(r >= 0.0 && r <= 1.0)) return ORACLE_BAD;
    const int g = n / n_groups;
    const int n_cached = (int)floor(r * (double)g);
    keyed *keys = (keyed *)malloc(sizeof(keyed) * (size_t)(g ? g : 1));
    if (!keys) return ORACLE_BAD;
    for (int grp = 0; grp < n_groups; ++grp) {
        for (int j = 0; j < g; ++j) { keys[j].m = metric[grp * g + j]; keys[j].i = grp * g + j; }
        qsort(keys, (size_t)g, sizeof(keyed), keyed_cmp);
        for (int j = 0; j < g; ++j) mask[keys[j].i] = (uint8_t)(j < n_cached ? 0 : 1);
    }
    free(keys);
    int32_t cnt = 0;
    for (int u = 0; u < n; ++u)
        if (mask[u]) idx[cnt++] = u;
    *n_active = cnt;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Compaction of the active units into what each destination would receive   */
/* (Section III-D, "Selective communication in TAPA"): message (src, dst)     */
/* carries src's active units, ascending, restricted to dst's heads; dst      */
/* concatenates the messages by source.  COMPACT = [P][H/P][n_active*T][D].   */
int oracle_pack_active(const uint16_t *x_seq, const int32_t *idx, int n_active, uint16_t *compact,
                       int P, int S, int H, int D, int T) {
    if (!shapes_ok(P, S, H, D) || T < 1 || (S / P) % T != 0) return ORACLE_BAD;
    const int Sl = S / P, Hl = H / P, units_per_rank = Sl / T;
    const size_t rows = (size_t)n_active * T; /* tokens per destination head */
    int a = 0;                                /* running slot over sources (ascending idx) */
    for (int src = 0; src < P; ++src) {
        /* the active units of this source are a contiguous run of idx */
        const int a0 = a;
        while (a < n_active && idx[a] / units_per_rank == src) ++a;
        const int cnt = a - a0;
        for (int dst = 0; dst < P; ++dst) {
            /* message[src][dst][unit][j][h_l][:] */
            uint16_t *message = (uint16_t *)malloc(2 * ((size_t)cnt * T * Hl * D + 1));
            if (!message) return ORACLE_BAD;
            for (int c = 0; c < cnt; ++c)
                for (int j = 0; j < T; ++j)
                    for (int hl = 0; hl < Hl; ++hl) {
                        const size_t tok = (size_t)idx[a0 + c] * T + j;
                        memcpy(message + (((size_t)c * T + j) * Hl + hl) * D,
                               x_seq + (tok * H + (size_t)dst * Hl + hl) * D, 2 * (size_t)D);
                    }
            /* receive side: slot a0 + c of every local head */
            for (int c = 0; c < cnt; ++c)
                for (int j = 0; j < T; ++j)
                    for (int hl = 0; hl < Hl; ++hl)
                        memcpy(compact + (((size_t)dst * Hl + hl) * rows + (size_t)(a0 + c) * T + j) * D,
                               message + (((size_t)c * T + j) * Hl + hl) * D, 2 * (size_t)D);
            free(message);
        }
    }
    return a == n_active ? ORACLE_OK : ORACLE_BAD; /* idx must be ascending */
}

/* Receiver-side reconstruction (Section III-D, "Post-Phase 2"): indexed      */
/* scatter of the active units over the cached head-parallel tensor; inactive */
/* rows keep their cached bits.                                               */
int oracle_unpack(const uint16_t *compact, const int32_t *idx, int n_active, uint16_t *cache_head,
                  int P, int S, int H, int D, int T) {
    if (!shapes_ok(P, S, H, D) || T < 1 || (S / P) % T != 0) return ORACLE_BAD;
    const size_t rows = (size_t)n_active * T;
    for (int h = 0; h < H; ++h)
        for (int a = 0; a < n_active; ++a)
            for (int j = 0; j < T; ++j)
                memcpy(cache_head + ((size_t)h * S + (size_t)idx[a] * T + j) * D,
                       compact + ((size_t)h * rows + (size_t)a * T + j) * D, 2 * (size_t)D);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Time-varying cache schedule (Section III-D, "Time-varying cache            */
/* scheduling").  Steps are numbered from 0.  (i) warm-up: the first `warmup`  */
/* steps run the full exchange; (ii) from the warm-up boundary on the cache    */
/* ratio r grows linearly from 0 (step `warmup`) to 1 (last step); (iii) every */
/* `sync_interval`-th step is a full exchange that resets the cache.           */
/* Reading: the paper gives no formula for the line nor the phase of the       */
/* periodic refresh; taken here as r = (t - w) / (T - 1 - w) and full steps    */
/* at t % interval == 0.                                                       */
int oracle_cache_schedule(int step, int total_steps, int warmup, int sync_interval,
                          int *full_exchange, double *r) {
    if (step < 0 || total_steps < 1 || step >= total_steps || warmup < 0 || sync_interval < 0) return ORACLE_BAD;
    int full = step < warmup;
    if (sync_interval > 0 && step % sync_interval == 0) full = 1;
    double ratio = 0.0;
    if (step >= warmup) {
        const int span = total_steps - 1 - warmup;
        ratio = span > 0 ? (double)(step - warmup) / (double)span : 0.0;
    }
    *full_exchange = full;
    *r = full ? 0.0 : ratio;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* The whole prologue of one layer, full exchange: V is exchanged first       */
/* (Section III-C), then Q and K after norm + RoPE.  Values do not depend on  */
/* the order of issue.  scratch must hold S*H*D uint16.                       */
int oracle_prologue(const uint16_t *q, const uint16_t *k, const uint16_t *v,
                    const uint16_t *wq, const uint16_t *wk, float eps, const float *cs,
                    int P, int S, int H, int D,
                    uint16_t *q_head, uint16_t *k_head, uint16_t *v_head, uint16_t *scratch) {
    int rc = oracle_ulysses_a2a(v, v_head, P, S, H, D);
    if (rc) return rc;
    rc = oracle_norm_rope(q, wq, eps, cs, S, H, D, scratch, NULL);
    if (rc) return rc;
    rc = oracle_ulysses_a2a(scratch, q_head, P, S, H, D);
    if (rc) return rc;
    rc = oracle_norm_rope(k, wk, eps, cs, S, H, D, scratch, NULL);
    if (rc) return rc;
    return oracle_ulysses_a2a(scratch, k_head, P, S, H, D);
}

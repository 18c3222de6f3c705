// Persistent layer-range kernel for passes of one or two rows.
//
// At one or two rows a decode step is nothing but a stream of weights from HBM (Sec. IV-B.3),
// and one kernel per projection leaves HBM idle at every kernel boundary.  This kernel runs a
// whole range of layers in ONE cooperative launch, one CTA per SM:
//
//   * warps 16..19 are producers.  They walk the same list of phases as everyone else but only
//     ever look at weights, which depend on nothing, so they keep TMA copies of [16 rows x 256
//     columns] weight boxes flowing into an 8-slot shared-memory ring across phase and layer
//     boundaries.  Producer p owns the ring slots p and p + 4 and cycles them on its own (one
//     thread needs a few hundred nanoseconds per copy, so four run side by side).  The ring is
//     what keeps HBM streaming while the consumers sit in a barrier or in the attention phases.
//     (Asking the L2 for weights further ahead was measured in three forms and lost each time:
//     tensor or bulk prefetches running ahead of the copies made every phase slower, gate/up by
//     30-80 %; a burst for the next gate/up bands during the attention phases delayed the
//     attention's own cache reads by as much as it later saved.)
//   * warps 0..15 are consumers.  Per layer they run six phases separated by grid-wide barriers:
//     RMSNorm + q/k/v + rotary embedding + cache append; attention partials; merge of the
//     splits; O-projection + residual; RMSNorm + gate/up + SiLU; down-projection + residual.
//     In a projection phase a CTA owns "bands" of 32 weight rows; warp w owns row w of each of
//     the band's two 16-row boxes (a rotary pair, a gate/up pair, or two plain rows), reads one
//     16-byte unit per lane per box, keeps fp32 sums across the whole inner dimension and
//     shuffles once per band.  Activations sit in shared memory as fp32, and the attention
//     output and the MLP activation travel between phases as fp32: at random initialisation a
//     rounding early in the stack is amplified by every later layer, and bf16 activations alone
//     put the exit states of a 28-layer stack 2-3 % from the fp64 reference.
//
// Every wait (ring slot, grid barrier) is bounded by a wall-clock limit; on a timeout the CTA
// raises ST_TIMEOUT, tells the other CTAs through the abort word, lets its copies land and
// returns.
#pragma once

#include "sparsk_attn.cuh"
#include "sparsk_gemm.cuh"

namespace sparsk {

constexpr int MK_CW = 16;                       // consumer warps
constexpr int MK_PW = 4;                        // producer warps
constexpr int MK_THREADS = (MK_CW + MK_PW) * 32;
constexpr int MK_BOX_ROWS = 16, MK_BOX_COLS = 256;
constexpr int MK_BOX_BYTES = MK_BOX_ROWS * MK_BOX_COLS * 2;  // 8 KB
constexpr int MK_SLOT_BYTES = 2 * MK_BOX_BYTES;              // two boxes per slot
constexpr int MK_SLOTS = 8;
constexpr int MK_MAX_ROWS = 4;
constexpr int MK_AREA_BYTES = 88 * 1024;        // shared memory behind the ring
constexpr int MK_ATT_WARPS = 3;                 // consumer warps that run attention items
constexpr int MK_ATT_NST = 2;
constexpr int MK_MAX_SPLITS = 32;             // the merge keeps one split per lane

// The area behind the ring holds the activations of a projection phase (M rows of bf16; when
// M rows of the whole inner dimension do not fit, a window of k-steps that is reloaded as the
// phase moves along), or the attention warps' query blocks and K/V rings.
inline size_t mk_attn_bytes(int head_dim)
{
    return (size_t)MK_ATT_WARPS * (16 * (head_dim + 8) * 2 + attn_warp_bytes(head_dim, MK_ATT_NST));
}
// k-steps of M fp32 activation rows that fit the area
__host__ __device__ inline int mk_act_window(int M) { return MK_AREA_BYTES / (M * MK_BOX_COLS * 4); }

enum { MKW_Q = 0, MKW_K, MKW_V, MKW_O, MKW_G, MKW_U, MKW_D, MKW_N };
enum { MK_QKV = 0, MK_ATTN = 1, MK_MERGE = 2, MK_OPROJ = 3, MK_GATEUP = 4, MK_DOWN = 5 };

// One layer's worth of what the phases need (device array, one entry per layer).
struct MkLayer {
    // per matrix (MKW_*): [16 rows x 256 columns] boxes without swizzle (passes of one or two rows),
    // then, MKW_N entries on, the same boxes as four 64-column blocks with the 128-byte swizzle
    // (view [64][rows][K/64], box {64, 16, 4}; passes of three and four rows read them with ldmatrix)
    CUtensorMap map[14];
    const bf16 *attn_gain, *mlp_gain;
    kv_t *kc, *vc;  // this layer's cache [slot][Hkv][S][hd]
};

struct MkArgs {
    const MkLayer *layers;       // device
    int layer_begin, layer_end;  // 0-based, [begin, end)
    float *h;                    // residual stream of the pass [rows][d]
    const int *row_slot, *row_pos, *grp_row0, *grp_nrows;
    int n_rows, n_groups;
    float *q_buf;                // [rows][Hq*hd]
    float *attn_o, *act;         // [rows][Hq*hd], [rows][F]
    float *part_o;
    float2 *part_ml;
    const float2 *rope;
    int d, Hq, Hkv, hd, F, S, n_slots;
    float eps;
    int att_splits, att_split_len;  // KV cut of the attention phase
    int att_qblk;                   // blocks of 16 query vectors per group
    unsigned long long *bar;        // grid barrier counter (monotonic)
    unsigned long long bar_base;    // its value when this launch starts
    int *abort_word;                // nonzero: some CTA gave up
    int *status;
    unsigned long long *trace;      // [1 + 6 * layers]: CTA 0's clock at the start and after every phase
};

__device__ __forceinline__ unsigned long long ld_acquire_u64(const unsigned long long *p)
{
    unsigned long long v;
    asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ int ld_volatile_i32(const int *p)
{
    int v;
    asm volatile("ld.volatile.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void mk_consumer_sync() { asm volatile("bar.sync 2, %0;" ::"n"(MK_CW * 32) : "memory"); }

// Bands and k-steps of a projection phase.
struct MkShape {
    int n_bands, k_steps;
};
__device__ __forceinline__ MkShape mk_shape(int type, const MkArgs &a)
{
    MkShape s;
    const int half = a.hd >> 1;
    switch (type) {
    case MK_QKV:
        s.n_bands = (a.Hq + a.Hkv) * (half / MK_BOX_ROWS) + (a.Hkv * a.hd + 2 * MK_BOX_ROWS - 1) / (2 * MK_BOX_ROWS);
        s.k_steps = (a.d + MK_BOX_COLS - 1) / MK_BOX_COLS;
        break;
    case MK_OPROJ:
        s.n_bands = (a.d + 2 * MK_BOX_ROWS - 1) / (2 * MK_BOX_ROWS);
        s.k_steps = (a.Hq * a.hd + MK_BOX_COLS - 1) / MK_BOX_COLS;
        break;
    case MK_GATEUP:
        s.n_bands = (a.F + MK_BOX_ROWS - 1) / MK_BOX_ROWS;
        s.k_steps = (a.d + MK_BOX_COLS - 1) / MK_BOX_COLS;
        break;
    case MK_DOWN:
        s.n_bands = (a.d + 2 * MK_BOX_ROWS - 1) / (2 * MK_BOX_ROWS);
        s.k_steps = (a.F + MK_BOX_COLS - 1) / MK_BOX_COLS;
        break;
    default:
        s.n_bands = 0;
        s.k_steps = 0;
    }
    return s;
}
// Descriptor and first row of the two boxes of band b.
__device__ __forceinline__ void mk_band(int type, const MkArgs &a, const MkLayer *L, int b, const CUtensorMap *(&map)[2],
                                        int (&row)[2])
{
    const int half = a.hd >> 1, per_head = half / MK_BOX_ROWS;
    switch (type) {
    case MK_QKV: {
        const int nq = a.Hq * per_head, nk = a.Hkv * per_head;
        if (b < nq + nk) {
            const bool isq = b < nq;
            const int bb = isq ? b : b - nq;
            map[0] = map[1] = &L->map[isq ? MKW_Q : MKW_K];
            row[0] = (bb / per_head) * a.hd + (bb % per_head) * MK_BOX_ROWS;
            row[1] = row[0] + half;
        } else {
            map[0] = map[1] = &L->map[MKW_V];
            row[0] = (b - nq - nk) * 2 * MK_BOX_ROWS;
            row[1] = row[0] + MK_BOX_ROWS;
        }
        break;
    }
    case MK_GATEUP:
        map[0] = &L->map[MKW_G];
        map[1] = &L->map[MKW_U];
        row[0] = row[1] = b * MK_BOX_ROWS;
        break;
    default:
        map[0] = map[1] = &L->map[type == MK_OPROJ ? MKW_O : MKW_D];
        row[0] = b * 2 * MK_BOX_ROWS;
        row[1] = row[0] + MK_BOX_ROWS;
    }
}

// This CTA's share of a projection phase, as segments (band, k-steps [ks0, ks1)).  q/k/v and
// gate/up deal whole bands round-robin (144 and F/16 bands fill 148 SMs well).  The two residual
// projections have d/32 bands, fewer than there are SMs, and an additive ending, so their
// (band, k-step) pairs are laid end to end and cut into equal contiguous shares; a share that
// ends inside a band adds its partial sums into the residual stream with atomics.
struct MkSeg {
    int band, ks0, ks1;
};
struct MkWalk {
    int k_steps, n_bands, j;
    bool stream;
    long pos, hi;
    __device__ void init(int type, const MkArgs &a)
    {
        const MkShape shp = mk_shape(type, a);
        k_steps = shp.k_steps;
        n_bands = shp.n_bands;
        stream = type == MK_OPROJ || type == MK_DOWN;
        j = blockIdx.x;
        const long T = (long)n_bands * k_steps;
        pos = (long)blockIdx.x * T / gridDim.x;
        hi = (long)(blockIdx.x + 1) * T / gridDim.x;
    }
    __device__ bool next(MkSeg &s)
    {
        if (stream) {
            if (pos >= hi) return false;
            s.band = (int)(pos / k_steps);
            s.ks0 = (int)(pos % k_steps);
            s.ks1 = (int)min((long)k_steps, s.ks0 + (hi - pos));
            pos += s.ks1 - s.ks0;
            return true;
        }
        if (j >= n_bands || k_steps < 1) return false;
        s.band = j;
        s.ks0 = 0;
        s.ks1 = k_steps;
        j += gridDim.x;
        return true;
    }
};

struct MkShared {
    uint64_t full[MK_SLOTS], empty[MK_SLOTS];
    int giving_up, never;
    int row_slot[MK_MAX_ROWS], row_pos[MK_MAX_ROWS], grp_row0[MK_MAX_ROWS], grp_nrows[MK_MAX_ROWS];  // copies of the row set
    float red[MK_CW];
    float red_rows[MK_MAX_ROWS][MK_CW];  // per-row partial sums of squares (tensor-core form: all rows at once)
};

// Consumers only: wait until every CTA has arrived at this barrier.
__device__ __forceinline__ bool mk_grid_barrier(const MkArgs &a, MkShared *sh, unsigned long long &epoch)
{
    mk_consumer_sync();
    epoch += gridDim.x;
    if (threadIdx.x == 0) {
        // release: everything this CTA wrote (ordered before by the CTA barrier) is visible to
        // whoever acquires the counter; no value comes back, so nothing waits on the round trip
        asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(a.bar), "l"(1ull) : "memory");
        unsigned long long t0 = 0;
        for (uint32_t spin = 0;; ++spin) {
            if (ld_acquire_u64(a.bar) >= epoch) break;
            if ((spin & 63u) == 63u) {
                if (ld_volatile_i32(a.abort_word) || sh->giving_up) {
                    // another CTA (or an earlier launch that was never cleaned up after) gave up:
                    // leave too, and say so, so that skipping the rest is never silent
                    sh->giving_up = 1;
                    atomicOr(a.status, ST_TIMEOUT);
                    break;
                }
                const unsigned long long now = global_ns();
                if (t0 == 0) t0 = now;
                else if (now - t0 > GM_TIMEOUT_NS) {
                    sh->giving_up = 1;
                    atomicOr(a.status, ST_TIMEOUT);
                    atomicExch(a.abort_word, 1);
                    break;
                }
            }
        }
        if (blockIdx.x == 0 && a.trace) a.trace[(epoch - a.bar_base) / gridDim.x] = global_ns();
    }
    mk_consumer_sync();
    return *(volatile int *)&sh->giving_up == 0;
}

}  // namespace sparsk

#include "sparsk_mega_phases.cuh"

// Persistent layer-range kernel for passes of 3..64 rows: the tcgen05 path without kernel
// boundaries.
//
// The per-layer sequence norm -> q/k/v GEMM -> finish -> attention -> merge -> O GEMM -> norm ->
// gate/up GEMM -> down GEMM is nine launches on the plain path, and at a few dozen rows each of
// them streams for 5-40 us while launch, prologue, ramp and drain cost 8-10 us.  Here the nine
// steps are phases of ONE cooperative kernel, one CTA per SM, separated by grid barriers:
//
//   warps 0..7   workers: norms, q/k/v finish, attention (two groups of four warps), merge, the
//                GEMM endings (warps 0..3 read TMEM), and the grid barrier
//   warp  8      issues tcgen05.mma for every ring item; owns the TMEM allocation
//   warps 9, 10  producers: TMA copies of weight tiles ([256 rows x 64] or two [128 x 64], 128-byte
//                swizzle) and of the activation tiles (hi and lo bf16 planes) into a four-slot ring
//
// Weights depend on nothing, so a producer copies the weight tile of an item as soon as its slot
// is free, also for items of a later phase; the activation tiles of an item wait until the grid
// barrier that completes their producer phase has been passed (the producers read the barrier
// counter themselves).  The attention phase uses the ring's shared memory, so no weight tile is
// copied before the barrier that ends the latest attention phase (a CTA without items in the
// phases in between would otherwise run ahead into it).  Waits are bounded as everywhere else.
//
// Off by default (option "tcmega"): at 64 rows its phases take 12 + 7 + 25..50 + 8..14 + 11 + 54 + 23
// us (q/k/v, finish, attention, merge, O, gate/up, down; plus 4-5 us per norm) against the
// launch-per-phase path's ~150 us per layer with programmatic dependent launch, because the ring
// that shares shared memory with the attention phase holds only four 32 KB weight tiles per SM.
// CTA 0 records its clock after every barrier (sparsk_phase_trace), which is how those phase
// times were measured.
#pragma once

#include "sparsk_attn.cuh"
#include "sparsk_gemm.cuh"
#include "sparsk_mega.cuh"

namespace sparsk {

constexpr int TK_SLOTS = 4;
constexpr int TK_PW = 2;        // producer warps; producer p owns slots p and p + 2
constexpr int TK_WORKERS = 8;   // worker warps
constexpr int TK_THREADS = (TK_WORKERS + 1 + TK_PW) * 32;
constexpr int TK_MAX_N = 64;    // rows per pass
constexpr int TK_A_BYTES = 2 * GM_BLK_BYTES;        // 32 KB of weights per item
constexpr int TK_B_BYTES = 2 * TK_MAX_N * GM_BK * 2;  // hi and lo tiles, 16 KB
constexpr int TK_ATT_BYTES = 104 * 1024;            // shared memory of one attention group
constexpr int TK_SMEM = 2 * TK_ATT_BYTES + 1024;    // >= ring (4 x 48 KB) + alignment slack

enum { TK_NORM_A = 0, TK_QKV, TK_FINISH, TK_ATTN, TK_MERGE, TK_OPROJ, TK_NORM_M, TK_GATEUP, TK_DOWN, TK_PHASES };

struct TkLayer {
    CUtensorMap wq, wk, wv, wo, wg, wu, wd;  // [64 x 256-row] boxes (gate/up: 128-row), 128-byte swizzle
    const bf16 *attn_gain, *mlp_gain;
    bf16 *kc, *vc;
};

struct TkArgs {
    CUtensorMap x_hi, x_lo, ao_hi, ao_lo, act_hi, act_lo;  // activation planes, [64 x box_n] boxes
    const TkLayer *layers;
    int layer_begin, layer_end;
    float *h;                                  // [rows][d]
    const int *row_slot, *row_pos, *grp_row0, *grp_nrows, *n_groups_dev;
    int m_rows, box_n;
    float *q32, *qkv_part;
    bf16 *x_hi_p, *x_lo_p, *ao_hi_p, *ao_lo_p, *act_hi_p, *act_lo_p;
    float *part_o;
    float2 *part_ml;
    const float2 *rope;
    int d, Hq, Hkv, hd, F, S, n_slots;
    float eps;
    int splits_qkv, splits_o, splits_down;     // cuts of the inner dimension per unit
    int att_groups, att_qblk, att_splits, att_split_len, att_mt;
    unsigned long long *bar;
    unsigned long long bar_base;
    int *abort_word, *status;
    unsigned long long *trace;                 // [1 + TK_PHASES * layers]: CTA 0's clock after every barrier
};

struct TkShared {
    uint64_t full_a[TK_SLOTS], full_b[TK_SLOTS], empty[TK_SLOTS], acc_full[2], acc_empty[2];
    uint32_t tmem_base;
    int giving_up, never;
    float red[8];
};

// Shape of a GEMM phase: inner dimension, units per matrix, cuts, pairing.
struct TkGemm {
    int K, units[3], splits, pair;
    __device__ int n_units() const { return (units[0] + (pair ? 0 : units[1] + units[2])) * splits; }
};
__device__ __forceinline__ TkGemm tk_gemm(int phase, const TkArgs &a)
{
    TkGemm g;
    const int qd = a.Hq * a.hd, kd = a.Hkv * a.hd;
    g.units[1] = g.units[2] = 0;
    g.pair = 0;
    switch (phase) {
    case TK_QKV:
        g.K = a.d; g.units[0] = (qd + 255) / 256; g.units[1] = g.units[2] = (kd + 255) / 256; g.splits = a.splits_qkv;
        break;
    case TK_OPROJ:
        g.K = qd; g.units[0] = (a.d + 255) / 256; g.splits = a.splits_o;
        break;
    case TK_GATEUP:
        g.K = a.d; g.units[0] = (a.F + 127) / 128; g.splits = 1; g.pair = 1;
        break;
    default:
        g.K = a.F; g.units[0] = (a.d + 255) / 256; g.splits = a.splits_down;
    }
    return g;
}
__device__ __forceinline__ bool tk_is_gemm(int phase)
{
    return phase == TK_QKV || phase == TK_OPROJ || phase == TK_GATEUP || phase == TK_DOWN;
}
// unit u of a GEMM phase -> (matrix, first row of accumulator 0, cut, k-block range)
__device__ __forceinline__ void tk_locate(const TkGemm &g, int u, int &mat, int &unit_row, int &sp, int &kb0, int &kb1)
{
    int t = u / g.splits;
    sp = u % g.splits;
    mat = 0;
    if (!g.pair) {
        if (t >= g.units[0]) { t -= g.units[0]; mat = 1; }
        if (mat == 1 && t >= g.units[1]) { t -= g.units[1]; mat = 2; }
    }
    unit_row = t * (g.pair ? GM_BM : 2 * GM_BM);
    const int kb_total = (g.K + GM_BK - 1) / GM_BK;
    kb0 = (int)((long)kb_total * sp / g.splits);
    kb1 = (int)((long)kb_total * (sp + 1) / g.splits);
}

__device__ __forceinline__ void tk_worker_sync() { asm volatile("bar.sync 3, %0;" ::"n"(TK_WORKERS * 32) : "memory"); }

// Workers only: arrive at the grid barrier and wait for everyone.
__device__ __forceinline__ bool tk_grid_barrier(const TkArgs &a, TkShared *sh, unsigned long long &epoch)
{
    asm volatile("fence.proxy.async;" ::: "memory");  // this phase's stores are read by other CTAs' TMA copies
    tk_worker_sync();
    epoch += gridDim.x;
    if (threadIdx.x == 0) {
        asm volatile("red.release.gpu.global.add.u64 [%0], %1;" ::"l"(a.bar), "l"(1ull) : "memory");
        unsigned long long t0 = 0;
        for (uint32_t spin = 0;; ++spin) {
            if (ld_acquire_u64(a.bar) >= epoch) break;
            if ((spin & 63u) == 63u) {
                if (ld_volatile_i32(a.abort_word) || sh->giving_up) {
                    sh->giving_up = 1;
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
    }
    tk_worker_sync();
    return *(volatile int *)&sh->giving_up == 0;
}

}  // namespace sparsk

#include "sparsk_tcmega_phases.cuh"
#include "sparsk_tcmega_kernel.cuh"

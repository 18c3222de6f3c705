// Batched weight-streaming path: Y^T = W X^T on the 5th-generation tensor cores.
//
// Once a pass has more than a handful of activation rows (a batch of sequences in the lower
// pass, pending + current rows of all full-depth sequences in the upper pass, a prompt chunk in
// prefill) every projection of a layer is a dense contraction whose weights must still be read
// from HBM exactly once (Sec. IV-B.3: one batched pass loads each weight matrix once).  The
// weights are therefore the M operand of tcgen05.mma (128 weight rows per tile, read through a
// 2-D TMA tensor map straight from the caller's row-major matrices), the active rows are the N
// operand (16..256, so a small batch still fills the instruction), accumulators live in TMEM.
//
// One persistent CTA per SM, three roles:
//   warp 0      producer: TMA loads of [128 x 64] weight tiles and [N x 64] activation tiles
//               (128-byte swizzle) into a ring of shared-memory stages
//   warp 1      issues tcgen05.mma for every stage, commits stages back to the producer and
//               finished accumulators to the epilogue; owns the TMEM allocation
//   warps 2..5  epilogue: tcgen05.ld of the accumulator (thread = weight row), then the
//               operation's own ending: rotary embedding + cache append, residual add,
//               SiLU(gate) * up, or logits + restricted arg max
// The activation operand is carried as two bf16 terms, x = hi + lo with lo = bf16(x - hi), and
// every weight tile is multiplied by both into the same accumulator: tcgen05 takes bf16 operands
// only, and at random initialisation a single bf16 rounding of the activations early in the
// stack is amplified by every later layer to 2-3 % at the exit of a 28-layer stack.  The second
// product costs tensor time and L2 traffic, not HBM bytes.
// Accumulators are double buffered in TMEM so a tile's epilogue overlaps the next tile's MMAs.
// Every wait is bounded: on a timeout the CTA raises ST_TIMEOUT, stops issuing work, drains its
// own copies, frees its TMEM and returns.
#pragma once

#include <cuda.h>

#include "sparsk_common.cuh"

namespace sparsk {

constexpr int GM_THREADS = 192;
constexpr int GM_BM = 128;                     // weight rows per accumulator (UMMA M)
constexpr int GM_BK = 64;                      // inner elements per k-block: one 128-byte swizzle span
constexpr int GM_MAX_N = 256;                  // activation rows per launch block (UMMA N limit)
constexpr int GM_BLK_BYTES = GM_BM * GM_BK * 2;  // one accumulator's weights for one k-block: 16 KB
constexpr int GM_MAX_STAGES = 6;
constexpr int GM_CHUNK = 16;                   // accumulator columns per epilogue chunk
constexpr int GM_XCHG_BYTES = GM_CHUNK * GM_BM * 4;
constexpr unsigned long long GM_TIMEOUT_NS = WAIT_TIMEOUT_NS;

// A unit of work is two accumulators of 128 weight rows each: either 256 consecutive rows of one
// matrix (one TMA box), or 128 rows of matrix 0 and the same 128 rows of matrix 1 ("pair": gate
// and up, whose results meet in the ending).  The TMA engine spends a fixed few hundred
// nanoseconds per copy whatever its size, so a stage is made of few, large boxes: with a
// three-dimensional view [64 elements][rows][K/64] of a row-major matrix one box carries two
// k-blocks of every row.
struct GemmArgs {
    int K;         // inner dimension
    int units[3];  // units of matrix 0, 1, 2 (pair: units[0] only)
    int row0[3];   // first row of each matrix that belongs to this product (a head's id range)
    int splits;    // cuts of the inner dimension per unit (> 1 only with an additive ending)
    int pair;      // 1: accumulator 1 comes from matrix 1
    int m_rows;    // activation rows of the whole launch; block y owns rows [256 y, 256 y + 256)
    int box_n;     // activation rows per TMA box (16, 32, 64, 128 or 256)
    int stages;    // ring depth
    int kb;        // k-blocks per stage (1 or 2)
    int three_d;   // 1: the descriptors are the [64][rows][K/64] views (needs K % 64 == 0)
    int *status;   // device status word
};

// (mbarrier, TMA and timer wrappers: sparsk_common.cuh)
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Shared-memory matrix descriptor of a K-major tile stored with the 128-byte swizzle: rows are
// 128 bytes, groups of eight rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_sw128(uint32_t smem_addr)
{
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) |
           (2ull << 61);
}
// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n.
__device__ __forceinline__ uint32_t umma_idesc_bf16(int n)
{
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(GM_BM >> 4) << 24);
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc, int accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t *bar)
{
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16])
{
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; i++) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void epi_barrier() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

// What an ending sees of one finished unit.
struct TileCtx {
    int matrix;      // which weight matrix the unit belongs to (0..2)
    int unit_row;    // first weight row of accumulator 0 inside that matrix (without GemmArgs::row0)
    int split;       // which cut of the inner dimension
    int row;         // this thread's row inside an accumulator (its TMEM lane), 0..127
    int m0, m_end;   // activation rows of this launch block: [m0, m_end)
    uint32_t taddr;  // TMEM address of accumulator 0, this thread's lane, column 0
    int acc_stride;  // columns between accumulator 0 and accumulator 1
    float *xchg;     // [GM_CHUNK][128] floats shared by the 128 epilogue threads
};

// ------------------------------------------------------------------ kernel
template <class Epi>
__global__ void __launch_bounds__(GM_THREADS, 1)
    wsgemm_kernel(const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
                  const __grid_constant__ CUtensorMap map_a2, const __grid_constant__ CUtensorMap map_b,
                  const __grid_constant__ CUtensorMap map_b_lo,
                  const GemmArgs g, const Epi epi)
{
    extern __shared__ __align__(1024) unsigned char gm_smem[];
    __shared__ __align__(8) uint64_t full_bar[GM_MAX_STAGES], empty_bar[GM_MAX_STAGES], acc_full[2], acc_empty[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int giving_up_s, never_s;
    volatile int *giving_up = &giving_up_s;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = (smem_u32(gm_smem) + 1023u) & ~1023u;  // swizzled tiles need 1024-byte alignment
    const int a_bytes = 2 * g.kb * GM_BLK_BYTES;                 // both accumulators' weights of a stage
    const int b_blk = g.box_n * GM_BK * 2;
    const int b_half = g.kb * b_blk;                              // the hi tiles; the lo tiles follow
    const int stage_bytes = a_bytes + 2 * b_half;
    // where accumulator a's rows of k-block j sit inside a stage
    const int a_blk_stride = g.pair ? GM_BLK_BYTES : 2 * GM_BLK_BYTES;
    const int a_acc_off = g.pair ? g.kb * GM_BLK_BYTES : GM_BLK_BYTES;
    float *xchg = reinterpret_cast<float *>(gm_smem + (ring - smem_u32(gm_smem)) + (size_t)g.stages * stage_bytes);

    const int m0 = blockIdx.y * GM_MAX_N;
    const int m_end = min(g.m_rows, m0 + GM_MAX_N);
    const int mma_n = ((m_end - m0) + 15) & ~15;
    const int kb_total = (g.K + GM_BK - 1) / GM_BK;
    const int k_stages = (kb_total + g.kb - 1) / g.kb;
    const int n_units = (g.units[0] + (g.pair ? 0 : g.units[1] + g.units[2])) * g.splits;
    // accumulator buffers: 2 when they fit, else 1
    const int acc_cols = 2 * mma_n;
    const int n_buf = (2 * acc_cols <= 512) ? 2 : 1;
    uint32_t alloc_cols = 32;
    while ((int)alloc_cols < n_buf * acc_cols) alloc_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < g.stages; s++) {
            mbar_init(&full_bar[s], 1);
            mbar_init(&empty_bar[s], 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(&acc_full[b], 1);
            mbar_init(&acc_empty[b], 4);
        }
        giving_up_s = 0;
        never_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)),
                     "r"(alloc_cols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;

    // Weights depend on no earlier kernel, activations and outputs do: the producer starts the
    // first weight copies before it waits for the grid dependency, the epilogue waits before it
    // touches anything, the MMA warp touches no global memory.
    griddep_launch();

    // unit u -> (matrix, first row, split)
    auto locate = [&](int u, int &mat, int &unit_row, int &sp) {
        int t = u / g.splits;
        sp = u % g.splits;
        mat = 0;
        if (!g.pair) {
            if (t >= g.units[0]) { t -= g.units[0]; mat = 1; }
            if (mat == 1 && t >= g.units[1]) { t -= g.units[1]; mat = 2; }
        }
        unit_row = t * (g.pair ? GM_BM : 2 * GM_BM);
    };

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // One thread needs a few hundred nanoseconds per TMA copy (barrier handshake included), so
        // the copies of a stage are issued by different lanes side by side: lane 0 waits for the
        // slot and posts the byte count, then lanes 0..2 each issue one box.
        uint32_t it = 0;
        bool ok = true;
        // pass 0 fills the ring's first round with weights only, then waits for the grid
        // dependency; pass 1 is the whole loop, adding only the activations to those stages
        for (int pass = 0; pass < 2 && ok; pass++) {
        it = 0;
        for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x) {
            int mat, unit_row, sp;
            locate(u, mat, unit_row, sp);
            const CUtensorMap *ma = mat == 0 ? &map_a0 : (mat == 1 ? &map_a1 : &map_a2);
            const int row = g.row0[mat] + unit_row;
            const int ks_beg = (int)((long)k_stages * sp / g.splits), ks_end = (int)((long)k_stages * (sp + 1) / g.splits);
            for (int ks = ks_beg; ks < ks_end; ks++, it++) {
                if (pass == 0 && it >= (uint32_t)g.stages) break;
                const bool early = it < (uint32_t)g.stages;  // its weights went out in pass 0
                const int s = it % g.stages;
                const uint32_t ph = (it / g.stages) & 1;
                int go = 1;
                if (lane == 0 && !(pass == 1 && early)) {
                    go = mbar_wait(&empty_bar[s], ph ^ 1, giving_up, g.status) ? 1 : 0;
                    if (go) mbar_expect_tx(&full_bar[s], (uint32_t)stage_bytes);
                }
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!(ok = go != 0)) break;
                const uint32_t st = ring + (uint32_t)s * stage_bytes;
                const int blk = ks * g.kb;
                // lane 0: accumulator 0's weights (or the whole 256-row box); lane 1: accumulator 1's
                // weights when they come from matrix 1; lanes 2 and 3: the two terms of the activations
                const CUtensorMap *mp = lane == 0 ? ma : (lane == 1 ? &map_a1 : (lane == 2 ? &map_b : &map_b_lo));
                const uint32_t dst = lane == 0 ? st : (lane == 1 ? st + a_acc_off : st + a_bytes + (lane == 3 ? b_half : 0));
                const int y = lane == 0 ? row : (lane == 1 ? g.row0[1] + unit_row : m0);
                const bool weights = lane == 0 || (lane == 1 && g.pair), acts = lane == 2 || lane == 3;
                if ((weights && !(pass == 1 && early)) || (acts && pass == 1)) {
                    if (g.three_d) tma_load_3d(dst, mp, &full_bar[s], 0, y, blk);
                    else tma_load_2d(dst, mp, &full_bar[s], blk * GM_BK, y);
                }
            }
            if (pass == 0 && it >= (uint32_t)g.stages) break;
        }
        if (pass == 0) griddep_wait();
        }
        if (!ok && lane == 0) {
            // giving up: let the copies already issued land (2 ms each at most) before the CTA
            // goes away; stage s was last filled in round (it - 1 - s) / stages
            for (int s = 0; s < g.stages; s++)
                if (it > (uint32_t)s) mbar_wait(&full_bar[s], ((it - 1 - s) / g.stages) & 1, &never_s, nullptr, 2000000ull);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(mma_n);
            uint32_t it = 0, unit_it = 0;
            bool ok = true;
            for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x, unit_it++) {
                const int sp = u % g.splits;
                const int ks_beg = (int)((long)k_stages * sp / g.splits), ks_end = (int)((long)k_stages * (sp + 1) / g.splits);
                const int buf = unit_it % n_buf;
                const uint32_t bph = (unit_it / n_buf) & 1;
                if (!(ok = mbar_wait(&acc_empty[buf], bph ^ 1, giving_up, g.status))) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * acc_cols);
                int accum = 0;
                for (int ks = ks_beg; ks < ks_end; ks++, it++) {
                    const int s = it % g.stages;
                    const uint32_t ph = (it / g.stages) & 1;
                    if (!(ok = mbar_wait(&full_bar[s], ph, giving_up, g.status))) break;
                    tc_fence_after();
                    const uint32_t a_addr = ring + (uint32_t)s * stage_bytes;
                    const uint32_t b_addr = a_addr + a_bytes;
                    for (int j = 0; j < g.kb; j++) {
                        if (ks * g.kb + j >= kb_total) break;  // a box's last k-block may lie outside K
#pragma unroll
                        for (int kk = 0; kk < GM_BK / 16; kk++) {
                            const uint64_t db = umma_desc_sw128(b_addr + j * b_blk + kk * 32);
                            const uint64_t dl = umma_desc_sw128(b_addr + b_half + j * b_blk + kk * 32);
                            const uint64_t da0 = umma_desc_sw128(a_addr + j * a_blk_stride + kk * 32);
                            const uint64_t da1 = umma_desc_sw128(a_addr + j * a_blk_stride + kk * 32 + a_acc_off);
                            umma_bf16(d0, da0, db, idesc, accum);
                            umma_bf16(d0, da0, dl, idesc, 1);
                            umma_bf16(d0 + mma_n, da1, db, idesc, accum);
                            umma_bf16(d0 + mma_n, da1, dl, idesc, 1);
                            accum = 1;
                        }
                    }
                    umma_commit(&empty_bar[s]);  // the stage is free once these MMAs have read it
                }
                if (ok) umma_commit(&acc_full[buf]);
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        griddep_wait();
        const int quad = warp & 3;  // TMEM lanes this warp may read: 32 quad .. 32 quad + 31
        TileCtx tc;
        tc.row = quad * 32 + lane;
        tc.m0 = m0;
        tc.m_end = m_end;
        tc.acc_stride = mma_n;
        tc.xchg = xchg;
        uint32_t unit_it = 0;
        bool ok = true;
        for (int u = blockIdx.x; u < n_units && ok; u += gridDim.x, unit_it++) {
            locate(u, tc.matrix, tc.unit_row, tc.split);
            const int buf = unit_it % n_buf;
            const uint32_t bph = (unit_it / n_buf) & 1;
            if (!(ok = mbar_wait(&acc_full[buf], bph, giving_up, g.status))) break;
            tc_fence_after();
            tc.taddr = tmem_base + ((uint32_t)(quad * 32) << 16) + (uint32_t)(buf * acc_cols);
            epi.tile(tc);
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&acc_empty[buf]);
        }
    }
    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(alloc_cols) : "memory");
    }
}

// ------------------------------------------------------------------ endings
// All endings walk an accumulator in chunks of 16 columns (activation rows); thread = weight row.

// q/k/v.  With the whole inner dimension in one unit: rotary embedding of q and k (pairs i,
// i + hd/2 sit hd/2 lanes apart, so values are exchanged through shared memory), q to the query
// buffer, k and v appended to the cache.  With the inner dimension cut across CTAs the partial
// sums are added into an fp32 scratch [rows][Hq*hd + 2*Hkv*hd] and qkv_finish_kernel does the rest.
struct QkvEnd {
    float *q_out;        // [rows][Hq*hd] fp32 (the attention kernels split it into two bf16 terms)
    kv_t *kc, *vc;       // this layer's cache [slot][Hkv][S][hd]
    const float2 *rope;  // [S][hd/2]
    const int *row_slot, *row_pos;
    float *partial;      // scratch for split sums, or NULL
    int Hq, Hkv, hd, S;

    __device__ void tile(const TileCtx &t) const
    {
        const int half = hd >> 1;
        const int n_rows_mat = (t.matrix == 0 ? Hq : Hkv) * hd;
        const int width = (Hq + 2 * Hkv) * hd;
        const int col0 = t.matrix == 0 ? 0 : (t.matrix == 1 ? Hq * hd : (Hq + Hkv) * hd);
        for (int a = 0; a < 2; a++) {
            const int n = t.unit_row + a * GM_BM + t.row;  // row inside its matrix
            const int head = n / hd, i = n % hd, j = i & (half - 1);
            const bool hi = i >= half;
            for (int c0 = 0; t.m0 + c0 < t.m_end; c0 += GM_CHUNK) {
                float v[GM_CHUNK];
                tmem_ld16(t.taddr + a * t.acc_stride + c0, v);
                if (partial) {
                    if (n < n_rows_mat) {
#pragma unroll
                        for (int c = 0; c < GM_CHUNK; c++) {
                            const int m = t.m0 + c0 + c;
                            if (m < t.m_end) atomicAdd(partial + (size_t)m * width + col0 + n, v[c]);
                        }
                    }
                    continue;
                }
                if (t.matrix < 2) {
#pragma unroll
                    for (int c = 0; c < GM_CHUNK; c++) t.xchg[c * GM_BM + t.row] = v[c];
                    epi_barrier();
                }
                if (n < n_rows_mat) {
#pragma unroll
                    for (int c = 0; c < GM_CHUNK; c++) {
                        const int m = t.m0 + c0 + c;
                        if (m >= t.m_end) break;
                        const int slot = row_slot[m], pos = row_pos[m];
                        if (t.matrix == 2) {
                            vc[(((size_t)slot * Hkv + head) * S + pos) * hd + i] = to_kv(v[c]);
                        } else {
                            const float other = t.xchg[c * GM_BM + (t.row ^ half)];
                            const float2 cs = rope[(size_t)pos * half + j];
                            const float r = hi ? v[c] * cs.x + other * cs.y : v[c] * cs.x - other * cs.y;
                            if (t.matrix == 0) q_out[(size_t)m * Hq * hd + n] = r;
                            else kc[(((size_t)slot * Hkv + head) * S + pos) * hd + i] = to_kv(r);
                        }
                    }
                }
                if (t.matrix < 2) epi_barrier();
            }
        }
    }
};

// Finishes a q/k/v product whose inner dimension was cut across CTAs: reads the summed row from
// the scratch, applies the rotary embedding, writes q and appends k, v to the cache, and clears
// the scratch for the next product.  One block per activation row.
static __global__ void __launch_bounds__(256) qkv_finish_kernel(float *__restrict__ partial, float *__restrict__ q_out,
                                                         kv_t *__restrict__ kc, kv_t *__restrict__ vc,
                                                         const float2 *__restrict__ rope,
                                                         const int *__restrict__ row_slot,
                                                         const int *__restrict__ row_pos, int n_rows, int Hq, int Hkv,
                                                         int hd, int S)
{
    griddep_launch();
    griddep_wait();
    const int m = blockIdx.x;
    if (m >= n_rows) return;
    const int half = hd >> 1, width = (Hq + 2 * Hkv) * hd;
    float *src = partial + (size_t)m * width;
    const int slot = row_slot[m], pos = row_pos[m];
    // q and k heads: one thread per rotary pair
    for (int p = threadIdx.x; p < (Hq + Hkv) * half; p += blockDim.x) {
        const int head = p / half, j = p % half;
        const float a = src[head * hd + j], b = src[head * hd + j + half];
        const float2 cs = rope[(size_t)pos * half + j];
        const float ra = a * cs.x - b * cs.y, rb = b * cs.x + a * cs.y;
        if (head < Hq) {
            float *dst = q_out + (size_t)m * Hq * hd + head * hd + j;
            dst[0] = ra;
            dst[half] = rb;
        } else {
            kv_t *dst = kc + (((size_t)slot * Hkv + (head - Hq)) * S + pos) * hd + j;
            dst[0] = to_kv(ra);
            dst[half] = to_kv(rb);
        }
    }
    for (int i = threadIdx.x; i < Hkv * hd; i += blockDim.x)
        vc[(((size_t)slot * Hkv + i / hd) * S + pos) * hd + i % hd] = to_kv(src[(Hq + Hkv) * hd + i]);
    __syncthreads();
    for (int i = threadIdx.x; i < width; i += blockDim.x) src[i] = 0.f;
}

// h[m][n] += (W x_m)[n]; with the inner dimension cut across CTAs the partial sums meet in h.
struct ResidEnd {
    float *h;  // [rows][n_out]
    int n_out, atomic;

    __device__ void tile(const TileCtx &t) const
    {
        for (int a = 0; a < 2; a++) {
            const int n = t.unit_row + a * GM_BM + t.row;
            for (int c0 = 0; t.m0 + c0 < t.m_end; c0 += GM_CHUNK) {
                float v[GM_CHUNK];
                tmem_ld16(t.taddr + a * t.acc_stride + c0, v);
                if (n >= n_out) continue;
#pragma unroll
                for (int c = 0; c < GM_CHUNK; c++) {
                    const int m = t.m0 + c0 + c;
                    if (m >= t.m_end) break;
                    float *dst = h + (size_t)m * n_out + n;
                    if (atomic) atomicAdd(dst, v[c]);
                    else *dst += v[c];
                }
            }
        }
    }
};

// u[m][f] = silu(gate) * up; accumulator 0 holds the gate rows, accumulator 1 the up rows.
struct GateUpEnd {
    bf16 *u, *u_lo;  // [rows][F]: u + u_lo carries the activation to 16 significant bits
    int F;

    __device__ void tile(const TileCtx &t) const
    {
        const int f = t.unit_row + t.row;
        for (int c0 = 0; t.m0 + c0 < t.m_end; c0 += GM_CHUNK) {
            float gt[GM_CHUNK], up[GM_CHUNK];
            tmem_ld16(t.taddr + c0, gt);
            tmem_ld16(t.taddr + t.acc_stride + c0, up);
            if (f >= F) continue;
#pragma unroll
            for (int c = 0; c < GM_CHUNK; c++) {
                const int m = t.m0 + c0 + c;
                if (m >= t.m_end) break;
                const float val = gt[c] / (1.f + __expf(-gt[c])) * up[c];
                const bf16 hi = __float2bfloat16(val);
                u[(size_t)m * F + f] = hi;
                u_lo[(size_t)m * F + f] = __float2bfloat16(val - __bfloat162float(hi));
            }
        }
    }
};

// Exit head over ids [lo, hi): per activation row the arg max (lowest id on ties) through the
// same packed 64-bit key the small-batch path uses; optional dump of the logits.
struct HeadEnd {
    const int *seq_of_row;
    unsigned long long *argmax;
    float *logits;  // optional [n_seq][V]
    int lo, hi, V;

    __device__ void tile(const TileCtx &t) const
    {
        const int lane = threadIdx.x & 31;
        for (int a = 0; a < 2; a++) {
            const int id = lo + t.unit_row + a * GM_BM + t.row;
            for (int c0 = 0; t.m0 + c0 < t.m_end; c0 += GM_CHUNK) {
                float v[GM_CHUNK];
                tmem_ld16(t.taddr + a * t.acc_stride + c0, v);
#pragma unroll
                for (int c = 0; c < GM_CHUNK; c++) {
                    const int m = t.m0 + c0 + c;
                    if (m >= t.m_end) break;  // uniform across the warp
                    unsigned long long key = id < hi ? argmax_key(v[c], id) : 0ull;
                    if (logits && id < hi) logits[(size_t)seq_of_row[m] * V + id] = v[c];
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        const unsigned long long other = __shfl_xor_sync(0xffffffffu, key, o);
                        key = other > key ? other : key;
                    }
                    if (lane == 0 && key) atomicMax(&argmax[seq_of_row[m]], key);
                }
            }
        }
    }
};

// RMSNorm of selected fp32 rows into the activation matrices the GEMM reads, as two bf16 terms:
// x + x_lo = h[row_idx ? row_idx[i] : i] / sqrt(mean(h^2) + eps) * gain.
static __global__ void __launch_bounds__(256) rmsnorm_rows_kernel(const float *__restrict__ h, const bf16 *__restrict__ gain,
                                                           const int *__restrict__ row_idx, bf16 *__restrict__ x,
                                                           bf16 *__restrict__ x_lo, int n_rows, int K, float eps)
{
    __shared__ float red[8];
    griddep_launch();
    griddep_wait();
    const int i = blockIdx.x;
    if (i >= n_rows) return;
    const float *src = h + (size_t)(row_idx ? row_idx[i] : i) * K;
    float ss = 0.f;
    for (int k = threadIdx.x * 4; k < K; k += 256 * 4) {
        const float4 v = *reinterpret_cast<const float4 *>(src + k);
        ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
    }
    ss = warp_sum(ss);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
    __syncthreads();
    float tot = 0.f;
#pragma unroll
    for (int w = 0; w < 8; w++) tot += red[w];
    const float inv = rsqrtf(tot / (float)K + eps);
    for (int k = threadIdx.x * 8; k < K; k += 256 * 8) {
        const float4 a = *reinterpret_cast<const float4 *>(src + k);
        const float4 b = *reinterpret_cast<const float4 *>(src + k + 4);
        float gn[8];
        unpack8(*reinterpret_cast<const uint4 *>(gain + k), gn);
        const float v[8] = {a.x * inv * gn[0], a.y * inv * gn[1], a.z * inv * gn[2], a.w * inv * gn[3],
                            b.x * inv * gn[4], b.y * inv * gn[5], b.z * inv * gn[6], b.w * inv * gn[7]};
        uint4 hi, lo;
        split8(v, hi, lo);
        *reinterpret_cast<uint4 *>(x + (size_t)i * K + k) = hi;
        *reinterpret_cast<uint4 *>(x_lo + (size_t)i * K + k) = lo;
    }
}

}  // namespace sparsk

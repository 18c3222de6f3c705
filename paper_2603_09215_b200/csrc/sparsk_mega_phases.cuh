// Phases of the persistent layer-range kernel (see sparsk_mega.cuh) and the kernel itself.
#pragma once

namespace sparsk {

// ------------------------------------------------------------------ activations -> shared memory
// Where column i (a multiple of 4) of a row sits inside the activation area.  A lane of a
// consumer warp needs the eight columns 8 lane .. 8 lane + 7 of a 256-column step (the columns of
// its 16-byte weight unit); read as two float4 at a 32-byte stride they would collide two ways on
// the banks, so each 256-column step is stored as two planes of 128 floats: columns 8 l + 0..3 at
// [4 l], columns 8 l + 4..7 at [128 + 4 l], and the two reads of a warp are both conflict-free.
__device__ __forceinline__ int mk_act_slot(int i)
{
    const int ci = i & (MK_BOX_COLS - 1);
    return (i - ci) + ((ci >> 2) & 1) * (MK_BOX_COLS / 2) + (ci >> 3) * 4;
}

// Columns [c0, c0 + ncols) of the M activation rows, as fp32, row m at act + m * ncols (in the
// layout of mk_act_slot).  With h:
// x = h / sqrt(mean(h^2) + eps) * gain; otherwise a copy of the fp32 rows x.  Columns at or
// beyond K are zeros (the last weight box is zero-filled there too).  ncols is a multiple of 256.
template <int M>
__device__ __forceinline__ void mk_load_act(float *act, int c0, int ncols, int K, const float *h, const float *x,
                                            const bf16 *gain, float eps, MkShared *sh)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int T = MK_CW * 32;
    mk_consumer_sync();  // everyone is done with what the area held
#pragma unroll
    for (int m = 0; m < M; m++) {
        float *dst = act + (size_t)m * ncols;
        if (h) {
            const float *src = h + (size_t)m * K;
            // a row that is loaded whole is parked in the area on its way through the sum of
            // squares and scaled in place afterwards: one trip to the L2 instead of two
            const bool whole = c0 == 0 && ncols >= K;
            float ss = 0.f;
            for (int i = tid * 4; i < (whole ? ncols : K); i += T * 4) {
                const float4 v = i < K ? *reinterpret_cast<const float4 *>(src + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
                if (whole) *reinterpret_cast<float4 *>(dst + mk_act_slot(i)) = v;
            }
            ss = warp_sum(ss);
            if (lane == 0) sh->red[warp] = ss;
            mk_consumer_sync();
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < MK_CW; w++) tot += sh->red[w];
            mk_consumer_sync();
            const float inv = rsqrtf(tot / (float)K + eps);
            if (whole) {
                for (int i = tid * 4; i < K; i += T * 4) {   // the thread's own float4s again
                    float4 *q = reinterpret_cast<float4 *>(dst + mk_act_slot(i));
                    const float4 p = *q;
                    const uint2 g2 = *reinterpret_cast<const uint2 *>(gain + i);
                    *q = make_float4(p.x * inv * bf_lo(g2.x), p.y * inv * bf_hi(g2.x), p.z * inv * bf_lo(g2.y),
                                     p.w * inv * bf_hi(g2.y));
                }
            } else {
                for (int i = tid * 4; i < ncols; i += T * 4) {
                    float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
                    const int k = c0 + i;
                    if (k < K) {
                        const float4 p = *reinterpret_cast<const float4 *>(src + k);
                        const uint2 g2 = *reinterpret_cast<const uint2 *>(gain + k);
                        o = make_float4(p.x * inv * bf_lo(g2.x), p.y * inv * bf_hi(g2.x), p.z * inv * bf_lo(g2.y),
                                        p.w * inv * bf_hi(g2.y));
                    }
                    *reinterpret_cast<float4 *>(dst + mk_act_slot(i)) = o;
                }
            }
        } else {
            const float *src = x + (size_t)m * K;
            for (int i = tid * 4; i < ncols; i += T * 4)
                *reinterpret_cast<float4 *>(dst + mk_act_slot(i)) =
                    c0 + i < K ? *reinterpret_cast<const float4 *>(src + c0 + i) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
    }
    mk_consumer_sync();
}

// ------------------------------------------------------------------ what a finished pair of sums becomes
// v0 = row `rib` of band b's first box, v1 = the same row of its second box (a rotary pair, a
// gate/up pair, or two plain rows), for activation row m.
__device__ __forceinline__ void mk_finish(int type, const MkArgs &a, const MkLayer *L, const MkShared *sh, int b, int rib,
                                          int m, float v0, float v1)
{
    const int half = a.hd >> 1, per_head = half / MK_BOX_ROWS;
    switch (type) {
    case MK_QKV: {
        const int nq = a.Hq * per_head, nk = a.Hkv * per_head;
        const int slot_id = sh->row_slot[m], pos = sh->row_pos[m];
        if (b < nq + nk) {
            const bool isq = b < nq;
            const int bb = isq ? b : b - nq;
            const int head = bb / per_head, i = (bb % per_head) * MK_BOX_ROWS + rib;
            const float2 cs = a.rope[(size_t)pos * half + i];
            const float ra = v0 * cs.x - v1 * cs.y, rb = v1 * cs.x + v0 * cs.y;
            if (isq) {
                float *dst = a.q_buf + (size_t)m * a.Hq * a.hd + head * a.hd + i;
                dst[0] = ra;
                dst[half] = rb;
            } else {
                kv_t *dst = L->kc + (((size_t)slot_id * a.Hkv + head) * a.S + pos) * a.hd + i;
                dst[0] = to_kv(ra);
                dst[half] = to_kv(rb);
            }
        } else {
            const int n0 = (b - nq - nk) * 2 * MK_BOX_ROWS + rib, n1 = n0 + MK_BOX_ROWS;
            const int kvd = a.Hkv * a.hd;
            if (n0 < kvd) L->vc[(((size_t)slot_id * a.Hkv + n0 / a.hd) * a.S + pos) * a.hd + n0 % a.hd] = to_kv(v0);
            if (n1 < kvd) L->vc[(((size_t)slot_id * a.Hkv + n1 / a.hd) * a.S + pos) * a.hd + n1 % a.hd] = to_kv(v1);
        }
        break;
    }
    case MK_GATEUP: {
        const int f = b * MK_BOX_ROWS + rib;
        if (f < a.F) a.act[(size_t)m * a.F + f] = v0 / (1.f + __expf(-v0)) * v1;
        break;
    }
    default: {
        const int n0 = b * 2 * MK_BOX_ROWS + rib, n1 = n0 + MK_BOX_ROWS;
        // shares of a band held by different CTAs meet in the residual stream
        if (n0 < a.d) atomicAdd(a.h + (size_t)m * a.d + n0, v0);
        if (n1 < a.d) atomicAdd(a.h + (size_t)m * a.d + n1, v1);
    }
    }
}

// ------------------------------------------------------------------ projection phase (consumers)
// The activations of the phase come from `h` (normalised with `gain`) or from the fp32 rows `x`,
// K columns each.  If M rows of the whole inner dimension fit the area they are loaded once;
// otherwise the area holds a window of k-steps that follows the CTA's segments.
template <int M>
__device__ __forceinline__ bool mk_project(int type, const MkArgs &a, const MkLayer *L, float *act, int K,
                                           const float *h, const float *x, const bf16 *gain, unsigned char *ring,
                                           MkShared *sh, uint32_t &it)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    MkWalk walk;
    walk.init(type, a);
    const int window = mk_act_window(M);
    const bool whole = walk.k_steps <= window;
    int win0 = 0, win1 = 0;  // k-steps the area holds: [win0, win1)
    if (whole) {
        win1 = walk.k_steps;
        mk_load_act<M>(act, 0, win1 * MK_BOX_COLS, K, h, x, gain, a.eps, sh);
    }
    const int ncols = whole ? walk.k_steps * MK_BOX_COLS : window * MK_BOX_COLS;
    MkSeg seg;
    while (walk.next(seg)) {
        const int b = seg.band;
        float acc[2][M];
#pragma unroll
        for (int r = 0; r < 2; r++)
#pragma unroll
            for (int m = 0; m < M; m++) acc[r][m] = 0.f;
        for (int ks = seg.ks0; ks < seg.ks1; ks++, it++) {
            if (ks < win0 || ks >= win1) {  // uniform across the CTA: move the window
                win0 = ks;
                win1 = min(walk.k_steps, ks + window);
                mk_load_act<M>(act, win0 * MK_BOX_COLS, ncols, K, h, x, gain, a.eps, sh);
            }
            const int s = it % MK_SLOTS;
            if (!mbar_wait(&sh->full[s], (it / MK_SLOTS) & 1, &sh->giving_up, a.status)) return false;
            const unsigned char *slot = ring + (size_t)s * MK_SLOT_BYTES + (size_t)warp * MK_BOX_COLS * 2 + lane * 16;
            float w0[8], w1[8];
            unpack8(*reinterpret_cast<const uint4 *>(slot), w0);
            unpack8(*reinterpret_cast<const uint4 *>(slot + MK_BOX_BYTES), w1);
#pragma unroll
            for (int m = 0; m < M; m++) {
                const float *xp = act + (size_t)m * ncols + (ks - win0) * MK_BOX_COLS + lane * 4;
                const float4 xa = *reinterpret_cast<const float4 *>(xp), xb = *reinterpret_cast<const float4 *>(xp + MK_BOX_COLS / 2);
                const float xv[8] = {xa.x, xa.y, xa.z, xa.w, xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                for (int j = 0; j < 8; j++) {
                    acc[0][m] = fmaf(w0[j], xv[j], acc[0][m]);
                    acc[1][m] = fmaf(w1[j], xv[j], acc[1][m]);
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->empty[s]);
        }
#pragma unroll
        for (int r = 0; r < 2; r++)
#pragma unroll
            for (int m = 0; m < M; m++) acc[r][m] = warp_sum(acc[r][m]);
        // lane m finishes activation row m
        float v0 = acc[0][0], v1 = acc[1][0];
#pragma unroll
        for (int m = 1; m < M; m++)
            if (lane == m) {
                v0 = acc[0][m];
                v1 = acc[1][m];
            }
        if (lane < M) mk_finish(type, a, L, sh, b, warp, lane, v0, v1);
    }
    return true;
}

// ------------------------------------------------------------------ three and four rows: tensor-core form
// With three or four activation rows the CUDA-core inner loop above is bound by shared-memory
// reads (every warp reads all rows' activations for its two weight rows).  Here a slot's two
// boxes arrive as four 64-column blocks each with the 128-byte swizzle, warp w takes box w / 8
// and the 32-column slice w % 8 of it, and multiplies with mma.sync m16n8k16: A = 16 weight rows
// x 16 columns (ldmatrix, conflict-free under the swizzle), B = 16 columns x 8 activation rows
// (rows beyond M are zeros), as two bf16 terms hi + lo of the activations (16 significant bits,
// as on the tcgen05 path).  The eight slices of a box meet in shared memory at the end of a band.
constexpr int MK_TC_RED_BYTES = 2 * 2 * 8 * 16 * 8 * 4;  // [parity][box][slice][16 rows][8 n] floats = 16 KB
__host__ __device__ inline int mk_tc_window(int M)
{
    return (MK_AREA_BYTES - MK_TC_RED_BYTES - 2 * M * 16) / (M * MK_BOX_COLS * 2 * 2);
}
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Columns [c0, c0 + ncols) of the M activation rows as two bf16 planes: hi at planes + m * rs,
// lo at planes + (M + m) * rs, rs = ncols + 8 elements (the padding spreads the rows over the
// banks).  Arithmetic as mk_load_act.
template <int M>
__device__ __forceinline__ void mk_load_act_tc(bf16 *planes, int c0, int ncols, int K, const float *h, const float *x,
                                               const bf16 *gain, float eps, MkShared *sh)
{
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int T = MK_CW * 32;
    const int rs = ncols + 8;
    mk_consumer_sync();  // everyone is done with what the area held
    float inv[M];
#pragma unroll
    for (int m = 0; m < M; m++) inv[m] = 1.f;
    if (h) {
        // the M rows' sums of squares side by side: one pass, one reduction
        float ss[M];
#pragma unroll
        for (int m = 0; m < M; m++) ss[m] = 0.f;
        for (int i = tid * 4; i < K; i += T * 4) {
#pragma unroll
            for (int m = 0; m < M; m++) {
                const float4 v = *reinterpret_cast<const float4 *>(h + (size_t)m * K + i);
                ss[m] += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
            }
        }
#pragma unroll
        for (int m = 0; m < M; m++) {
            ss[m] = warp_sum(ss[m]);
            if (lane == 0) sh->red_rows[m][warp] = ss[m];
        }
        mk_consumer_sync();
#pragma unroll
        for (int m = 0; m < M; m++) {
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < MK_CW; w++) tot += sh->red_rows[m][w];
            inv[m] = rsqrtf(tot / (float)K + eps);
        }
    }
    // all rows in one flat loop, so that the loads of several rows are in flight together
    const float *src = h ? h : x;
    const int per_row = ncols / 4;
#pragma unroll 4
    for (int idx = tid; idx < M * per_row; idx += T) {
        const int m = idx / per_row, i = (idx - m * per_row) * 4;
        float4 o = make_float4(0.f, 0.f, 0.f, 0.f);
        const int k = c0 + i;
        if (k < K) {
            o = *reinterpret_cast<const float4 *>(src + (size_t)m * K + k);
            if (h) {
                const uint2 g2 = *reinterpret_cast<const uint2 *>(gain + k);
                float sc = inv[0];
#pragma unroll
                for (int q = 1; q < M; q++)
                    if (m == q) sc = inv[q];
                o = make_float4(o.x * sc * bf_lo(g2.x), o.y * sc * bf_hi(g2.x), o.z * sc * bf_lo(g2.y), o.w * sc * bf_hi(g2.y));
            }
        }
        uint2 hi, lo;
        split_pair(o.x, o.y, hi.x, lo.x);
        split_pair(o.z, o.w, hi.y, lo.y);
        *reinterpret_cast<uint2 *>(planes + (size_t)m * rs + i) = hi;
        *reinterpret_cast<uint2 *>(planes + (size_t)(M + m) * rs + i) = lo;
    }
    mk_consumer_sync();
}

template <int M>
__device__ __forceinline__ bool mk_project_tc(int type, const MkArgs &a, const MkLayer *L, unsigned char *area, int K,
                                              const float *h, const float *x, const bf16 *gain, unsigned char *ring,
                                              MkShared *sh, uint32_t &it)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int box = warp >> 3, slice = warp & 7;
    bf16 *planes = reinterpret_cast<bf16 *>(area);
    float *red = reinterpret_cast<float *>(area + MK_AREA_BYTES - MK_TC_RED_BYTES);
    MkWalk walk;
    walk.init(type, a);
    const int window = mk_tc_window(M);
    const bool whole = walk.k_steps <= window;
    int win0 = 0, win1 = 0;  // k-steps the area holds: [win0, win1)
    const int ncols = whole ? walk.k_steps * MK_BOX_COLS : window * MK_BOX_COLS;
    const int rs = ncols + 8;
    if (whole) {
        win1 = walk.k_steps;
        mk_load_act_tc<M>(planes, 0, ncols, K, h, x, gain, a.eps, sh);
    }
    // this lane's row address inside a 64-column block for ldmatrix: matrices (rows 0-7, k 0-7),
    // (rows 8-15, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15)
    const int lrow = (lane & 7) + ((lane >> 3) & 1) * 8, lchk = lane >> 4;
    const uint32_t a_off = (uint32_t)box * MK_BOX_BYTES + (uint32_t)(slice >> 1) * (MK_BOX_ROWS * 128) + (uint32_t)lrow * 128;
    MkSeg seg;
    uint32_t band_it = 0;
    while (walk.next(seg)) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        for (int ks = seg.ks0; ks < seg.ks1; ks++, it++) {
            if (ks < win0 || ks >= win1) {  // uniform across the CTA: move the window
                win0 = ks;
                win1 = min(walk.k_steps, ks + window);
                mk_load_act_tc<M>(planes, win0 * MK_BOX_COLS, ncols, K, h, x, gain, a.eps, sh);
            }
            const int s = it % MK_SLOTS;
            if (!mbar_wait(&sh->full[s], (it / MK_SLOTS) & 1, &sh->giving_up, a.status)) return false;
            const uint32_t slot = smem_u32(ring) + (uint32_t)s * MK_SLOT_BYTES + a_off;
            const bf16 *bp = planes + (size_t)g * rs + (ks - win0) * MK_BOX_COLS + slice * 32 + 2 * t;
#pragma unroll
            for (int j = 0; j < 2; j++) {
                uint32_t af[4];
                const uint32_t chunk = (uint32_t)((slice & 1) * 4 + j * 2 + lchk);
                asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                             : "=r"(af[0]), "=r"(af[1]), "=r"(af[2]), "=r"(af[3])
                             : "r"(slot + ((chunk ^ (uint32_t)(lrow & 7)) << 4)));
                uint32_t b0 = 0, b1 = 0, c0 = 0, c1 = 0;
                if (g < M) {
                    b0 = *reinterpret_cast<const uint32_t *>(bp + j * 16);
                    b1 = *reinterpret_cast<const uint32_t *>(bp + j * 16 + 8);
                    c0 = *reinterpret_cast<const uint32_t *>(bp + (size_t)M * rs + j * 16);
                    c1 = *reinterpret_cast<const uint32_t *>(bp + (size_t)M * rs + j * 16 + 8);
                }
                mma_bf16_16816(acc, af, b0, b1);
                mma_bf16_16816(acc, af, c0, c1);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->empty[s]);
        }
        // the eight slices of each box meet: [parity][box][slice][16 rows][8 n]
        float *mine = red + ((((band_it & 1) * 2 + box) * 8 + slice) * 16) * 8;
        *reinterpret_cast<float2 *>(mine + g * 8 + 2 * t) = make_float2(acc[0], acc[1]);
        *reinterpret_cast<float2 *>(mine + (g + 8) * 8 + 2 * t) = make_float2(acc[2], acc[3]);
        mk_consumer_sync();
        if (threadIdx.x < MK_BOX_ROWS * M) {
            const int rib = threadIdx.x / M, m = threadIdx.x % M;
            const float *r0 = red + (((band_it & 1) * 2 + 0) * 8 * 16) * 8 + rib * 8 + m;
            const float *r1 = red + (((band_it & 1) * 2 + 1) * 8 * 16) * 8 + rib * 8 + m;
            float v0 = 0.f, v1 = 0.f;
#pragma unroll
            for (int sl = 0; sl < 8; sl++) {
                v0 += r0[sl * 16 * 8];
                v1 += r1[sl * 16 * 8];
            }
            mk_finish(type, a, L, sh, seg.band, rib, m, v0, v1);
        }
        band_it++;
    }
    return true;
}

// One or two rows: CUDA-core form with fp32 activations; three and four: tensor-core form.
template <int M>
__device__ __forceinline__ bool mk_proj(int type, const MkArgs &a, const MkLayer *L, unsigned char *area, int K,
                                        const float *h, const float *x, const bf16 *gain, unsigned char *ring, MkShared *sh,
                                        uint32_t &it)
{
    if (M >= 3) return mk_project_tc<M>(type, a, L, area, K, h, x, gain, ring, sh, it);
    return mk_project<M>(type, a, L, reinterpret_cast<float *>(area), K, h, x, gain, ring, sh, it);
}

}  // namespace sparsk

#include "sparsk_mega_attn.cuh"
#include "sparsk_mega_kernel.cuh"

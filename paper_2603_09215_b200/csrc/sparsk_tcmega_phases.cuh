// Worker phases of the persistent tcgen05 layer kernel (see sparsk_tcmega.cuh).  All eight worker
// warps (256 threads) call each phase; rows or items are dealt round-robin over the CTAs.
#pragma once

namespace sparsk {

// x_hi + x_lo = RMSNorm(h[r]) * gain for the pass's rows (the arithmetic of rmsnorm_rows_kernel).
__device__ __forceinline__ void tk_norm(const TkArgs &a, const bf16 *gain, TkShared *sh)
{
    const int tid = threadIdx.x, K = a.d;
    for (int r = blockIdx.x; r < a.m_rows; r += gridDim.x) {
        const float *src = a.h + (size_t)r * K;
        float ss = 0.f;
        for (int k = tid * 4; k < K; k += TK_WORKERS * 32 * 4) {
            const float4 v = *reinterpret_cast<const float4 *>(src + k);
            ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
        }
        ss = warp_sum(ss);
        if ((tid & 31) == 0) sh->red[tid >> 5] = ss;
        tk_worker_sync();
        float tot = 0.f;
#pragma unroll
        for (int w = 0; w < TK_WORKERS; w++) tot += sh->red[w];
        tk_worker_sync();
        const float inv = rsqrtf(tot / (float)K + a.eps);
        for (int k = tid * 8; k < K; k += TK_WORKERS * 32 * 8) {
            const float4 p = *reinterpret_cast<const float4 *>(src + k);
            const float4 q = *reinterpret_cast<const float4 *>(src + k + 4);
            float gn[8];
            unpack8(*reinterpret_cast<const uint4 *>(gain + k), gn);
            const float v[8] = {p.x * inv * gn[0], p.y * inv * gn[1], p.z * inv * gn[2], p.w * inv * gn[3],
                                q.x * inv * gn[4], q.y * inv * gn[5], q.z * inv * gn[6], q.w * inv * gn[7]};
            uint4 hi, lo;
            split8(v, hi, lo);
            *reinterpret_cast<uint4 *>(a.x_hi_p + (size_t)r * K + k) = hi;
            *reinterpret_cast<uint4 *>(a.x_lo_p + (size_t)r * K + k) = lo;
        }
    }
}

// Finishes the q/k/v product whose partial sums sit in the fp32 scratch: rotary embedding, q to
// the query buffer, k and v appended to the cache, scratch cleared (as qkv_finish_kernel).
__device__ __forceinline__ void tk_qkv_finish(const TkArgs &a, const TkLayer *L)
{
    const int tid = threadIdx.x, hd = a.hd, half = hd >> 1, Hq = a.Hq, Hkv = a.Hkv;
    const int width = (Hq + 2 * Hkv) * hd;
    for (int m = blockIdx.x; m < a.m_rows; m += gridDim.x) {
        float *src = a.qkv_part + (size_t)m * width;
        const int slot = a.row_slot[m], pos = a.row_pos[m];
        for (int p = tid; p < (Hq + Hkv) * half; p += TK_WORKERS * 32) {
            const int head = p / half, j = p % half;
            const float x = src[head * hd + j], y = src[head * hd + j + half];
            const float2 cs = a.rope[(size_t)pos * half + j];
            const float ra = x * cs.x - y * cs.y, rb = y * cs.x + x * cs.y;
            if (head < Hq) {
                float *dst = a.q32 + (size_t)m * Hq * hd + head * hd + j;
                dst[0] = ra;
                dst[half] = rb;
            } else {
                bf16 *dst = L->kc + (((size_t)slot * Hkv + (head - Hq)) * a.S + pos) * hd + j;
                dst[0] = __float2bfloat16(ra);
                dst[half] = __float2bfloat16(rb);
            }
        }
        for (int i = tid; i < Hkv * hd; i += TK_WORKERS * 32)
            L->vc[(((size_t)slot * Hkv + i / hd) * a.S + pos) * hd + i % hd] = __float2bfloat16(src[(Hq + Hkv) * hd + i]);
        tk_worker_sync();
        for (int i = tid; i < width; i += TK_WORKERS * 32) src[i] = 0.f;
    }
}

// Attention partials: the two four-warp groups of a CTA each run attn_partial_body over virtual
// block indices (group * n_qblk + query block, kv head, split), with their own shared memory and
// their own named barrier.
struct TkGroupSync {
    int id;
    __device__ void operator()() const { asm volatile("bar.sync %0, 128;" ::"r"(id) : "memory"); }
};
template <int HD>
__device__ __forceinline__ void tk_attention(const TkArgs &a, const TkLayer *L, unsigned char *smem)
{
    AttnArgs at;
    at.q = nullptr; at.q32 = a.q32; at.kc = L->kc; at.vc = L->vc;
    at.grp_row0 = a.grp_row0; at.grp_nrows = a.grp_nrows; at.row_slot = a.row_slot; at.row_pos = a.row_pos;
    at.n_groups = a.n_groups_dev;
    at.part_o = a.part_o; at.part_ml = a.part_ml; at.out = a.ao_hi_p; at.out_lo = a.ao_lo_p;
    at.Hq = a.Hq; at.Hkv = a.Hkv; at.S = a.S; at.n_qblk = a.att_qblk; at.n_splits = a.att_splits;
    at.split_len = a.att_split_len; at.n_slots = a.n_slots; at.n_rows = a.m_rows;
    at.nq_min = 0; at.nq_max = 1 << 30;
    const int grp = threadIdx.x >> 7, tid = threadIdx.x & 127;
    unsigned char *my = smem + (size_t)grp * TK_ATT_BYTES;
    const TkGroupSync sync{4 + grp};
    const int nx = a.att_groups * a.att_qblk, n_virtual = nx * a.Hkv * a.att_splits;
    for (int v = blockIdx.x * 2 + grp; v < n_virtual; v += gridDim.x * 2) {
        const int bx = v % nx, hk = (v / nx) % a.Hkv, sp = v / (nx * a.Hkv);
        sync();  // the group is done with the previous item's shared memory
        if (a.att_mt == 2) attn_partial_body<HD, 2, 2>(at, bx, hk, sp, my, tid, sync);
        else attn_partial_body<HD, 1, 2>(at, bx, hk, sp, my, tid, sync);
    }
}

// Merge of the splits into the two bf16 planes of the attention output (as attn_merge_kernel);
// items (row, head), HD threads each, two items per CTA at a time.
template <int HD>
__device__ __forceinline__ void tk_merge(const TkArgs &a)
{
    constexpr int PER = TK_WORKERS * 32 / HD;  // items a CTA handles side by side
    const int sub = threadIdx.x / HD, t = threadIdx.x % HD;
    const int n_items = a.m_rows * a.Hq;
    if (sub >= PER) return;
    for (int item = blockIdx.x * PER + sub; item < n_items; item += gridDim.x * PER) {
        const size_t cell0 = (size_t)item * a.att_splits;
        float M = -INFINITY;
        for (int s = 0; s < a.att_splits; s++) M = fmaxf(M, a.part_ml[cell0 + s].x);
        float den = 0.f, num = 0.f;
        for (int s = 0; s < a.att_splits; s++) {
            const float2 ml = a.part_ml[cell0 + s];
            if (ml.x == -INFINITY) continue;
            const float w = __expf(ml.x - M);
            den += ml.y * w;
            num += a.part_o[(cell0 + s) * HD + t] * w;
        }
        const float val = den > 0.f ? num / den : 0.f;
        const bf16 hi = __float2bfloat16(val);
        a.ao_hi_p[(size_t)item * HD + t] = hi;
        a.ao_lo_p[(size_t)item * HD + t] = __float2bfloat16(val - __bfloat162float(hi));
    }
}

}  // namespace sparsk

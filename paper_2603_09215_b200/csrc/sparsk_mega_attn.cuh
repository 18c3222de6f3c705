// Attention and split-merge phases of the persistent layer-range kernel (see sparsk_mega.cuh).
#pragma once

namespace sparsk {

// Items (group, query block, kv head, split) are dealt to MK_ATT_WARPS warps of every CTA; a warp
// runs its item alone: 16 query vectors (query heads of the kv head, for the group's rows), its
// own two-stage K/V ring inside the activation area, one partial per item.  The arithmetic is
// that of attn_partial_kernel with one m16 tile (queries and softmax weights as two fp16 terms).
template <int HD>
__device__ __forceinline__ void mk_attention(const MkArgs &a, const MkLayer *L, unsigned char *area, const MkShared *sh)
{
    constexpr int KP = HD + 8, CH = HD / 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (warp >= MK_ATT_WARPS) return;
    // per warp: its 16 query vectors (hi and lo term), then the K/V ring
    kv_t *Qs = reinterpret_cast<kv_t *>(area) + (size_t)warp * (2 * 16 + MK_ATT_NST * 2 * AT_TP) * KP;
    kv_t *Ql = Qs + 16 * KP;
    kv_t *wr = Ql + 16 * KP;
    const int G = a.Hq / a.Hkv;
    const int n_workers = gridDim.x * MK_ATT_WARPS, worker = warp * gridDim.x + blockIdx.x;
    const int n_qblk = a.att_qblk;
    const int n_items = a.n_groups * n_qblk * a.Hkv * a.att_splits;
    const float scale = rsqrtf((float)HD);
    for (int item = worker; item < n_items; item += n_workers) {
        int t = item;
        const int sp = t % a.att_splits; t /= a.att_splits;
        const int hk = t % a.Hkv; t /= a.Hkv;
        const int qb = t % n_qblk, g = t / n_qblk;
        const int row0 = sh->grp_row0[g], nrows = sh->grp_nrows[g];
        const int nq = nrows * G, q0 = qb * 16;
        if (row0 < 0 || nrows < 1 || row0 + nrows > a.n_rows || q0 >= nq) continue;
        const int nq_here = min(16, nq - q0);
        const int slot = sh->row_slot[row0], pos0 = sh->row_pos[row0];
        const bool sane = slot >= 0 && slot < a.n_slots && pos0 >= 0;
        const int last_row = (q0 + nq_here - 1) / G;
        const int kv_end_all = sane ? min(pos0 + last_row + 1, a.S) : 0;
        const int w_beg = sp * a.att_split_len;
        const int w_end = min(w_beg + a.att_split_len, kv_end_all);
        const int n_tiles = w_end > w_beg ? (w_end - w_beg + AT_TP - 1) / AT_TP : 0;
        const kv_t *kbase = L->kc + ((size_t)(sane ? slot : 0) * a.Hkv + hk) * a.S * HD;
        const kv_t *vbase = L->vc + ((size_t)(sane ? slot : 0) * a.Hkv + hk) * a.S * HD;

        auto issue = [&](int tt) {
            kv_t *kt = wr + (size_t)(tt % MK_ATT_NST) * 2 * AT_TP * KP, *vt = kt + AT_TP * KP;
            const int p0 = w_beg + tt * AT_TP;
#pragma unroll
            for (int i = lane; i < AT_TP * CH; i += 32) {
                const int r = i / CH, c = i % CH;
                const bool ok = p0 + r < w_end;  // rows past the end are zero-filled
                const size_t off = (size_t)(ok ? p0 + r : w_beg) * HD + c * 8;
                cp_async16(&kt[r * KP + c * 8], kbase + off, ok ? 16 : 0);
                cp_async16(&vt[r * KP + c * 8], vbase + off, ok ? 16 : 0);
            }
        };
        float o[HD / 8][4], m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
        for (int nt = 0; nt < HD / 8; nt++)
#pragma unroll
            for (int e = 0; e < 4; e++) o[nt][e] = 0.f;
        int limit[2];
#pragma unroll
        for (int hf = 0; hf < 2; hf++) {
            const int qi = (lane >> 2) + hf * 8;
            limit[hf] = qi < nq_here ? pos0 + (q0 + qi) / G : -1;
        }
        if (n_tiles > 0) issue(0);
        cp_async_commit();
        if (n_tiles > 1) issue(1);
        cp_async_commit();
        // the queries, while the first tiles are on their way
        __syncwarp();
        for (int i = lane; i < 16 * CH; i += 32) {
            const int qi = i / CH, c = i % CH;
            uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
            if (qi < nq_here) {
                const int qg = q0 + qi, r = qg / G, j = qg % G;
                const float *src = a.q_buf + (size_t)(row0 + r) * a.Hq * HD + (hk * G + j) * HD + c * 8;
                const float4 x0 = *reinterpret_cast<const float4 *>(src), x1 = *reinterpret_cast<const float4 *>(src + 4);
                const float v[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                split8_h(v, hi, lo);
            }
            *reinterpret_cast<uint4 *>(&Qs[qi * KP + c * 8]) = hi;
            *reinterpret_cast<uint4 *>(&Ql[qi * KP + c * 8]) = lo;
        }
        __syncwarp();

        for (int tt = 0; tt < n_tiles; tt++) {
            cp_async_wait<1>();  // all but the newest group: tile tt has landed
            __syncwarp();
            const kv_t *Kt = wr + (size_t)(tt % MK_ATT_NST) * 2 * AT_TP * KP, *Vt = Kt + AT_TP * KP;
            const int p0 = w_beg + tt * AT_TP;
            float s[2][4];
#pragma unroll
            for (int nt = 0; nt < 2; nt++)
#pragma unroll
                for (int e = 0; e < 4; e++) s[nt][e] = 0.f;
#pragma unroll
            for (int ks = 0; ks < HD / 16; ks++) {
                uint32_t kb[4], qa[4], ql[4];
                ldsm_x4(kb, &Kt[((lane & 7) + ((lane >> 4) << 3)) * KP + ks * 16 + ((lane >> 3) & 1) * 8]);
                ldsm_x4(qa, &Qs[((lane & 7) + ((lane >> 3) & 1) * 8) * KP + ks * 16 + (lane >> 4) * 8]);
                ldsm_x4(ql, &Ql[((lane & 7) + ((lane >> 3) & 1) * 8) * KP + ks * 16 + (lane >> 4) * 8]);
                mma_f16(s[0], qa, kb[0], kb[1]);
                mma_f16(s[1], qa, kb[2], kb[3]);
                mma_f16(s[0], ql, kb[0], kb[1]);
                mma_f16(s[1], ql, kb[2], kb[3]);
            }
            uint32_t pa[4], pl[4];
#pragma unroll
            for (int hf = 0; hf < 2; hf++) {
                float v[4];
                float tmax = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 2; nt++)
#pragma unroll
                    for (int e = 0; e < 2; e++) {
                        const int p = p0 + nt * 8 + (lane & 3) * 2 + e;
                        const bool ok = p < w_end && p <= limit[hf];
                        v[nt * 2 + e] = ok ? s[nt][hf * 2 + e] * scale : -INFINITY;
                        tmax = fmaxf(tmax, v[nt * 2 + e]);
                    }
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
                const float m_new = fmaxf(m_run[hf], tmax);
                float alpha = 1.f, psum = 0.f;
                if (m_new != -INFINITY) {
                    alpha = __expf(m_run[hf] - m_new);
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        v[i] = __expf(v[i] - m_new);
                        psum += v[i];
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 4; i++) v[i] = 0.f;
                }
                l_run[hf] = l_run[hf] * alpha + psum;
                m_run[hf] = m_new;
                split_pair_h(v[0], v[1], pa[hf], pl[hf]);
                split_pair_h(v[2], v[3], pa[2 + hf], pl[2 + hf]);
#pragma unroll
                for (int nt = 0; nt < HD / 8; nt++) {
                    o[nt][hf * 2] *= alpha;
                    o[nt][hf * 2 + 1] *= alpha;
                }
            }
#pragma unroll
            for (int np = 0; np < HD / 16; np++) {
                uint32_t vb[4];
                ldsm_x4_t(vb, &Vt[((lane & 7) + ((lane >> 3) & 1) * 8) * KP + np * 16 + (lane >> 4) * 8]);
                mma_f16(o[2 * np], pa, vb[0], vb[1]);
                mma_f16(o[2 * np + 1], pa, vb[2], vb[3]);
                mma_f16(o[2 * np], pl, vb[0], vb[1]);
                mma_f16(o[2 * np + 1], pl, vb[2], vb[3]);
            }
            __syncwarp();  // everyone is done with this stage: refill it with the tile after next
            if (tt + 2 < n_tiles) issue(tt + 2);
            cp_async_commit();
        }
        cp_async_wait<0>();
        // this item's partial
#pragma unroll
        for (int hf = 0; hf < 2; hf++) {
            float l = l_run[hf];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int qi = (lane >> 2) + hf * 8;
            if (qi < nq_here) {
                const int qg = q0 + qi, r = qg / G, j = qg % G;
                const size_t cell = ((size_t)(row0 + r) * a.Hq + hk * G + j) * a.att_splits + sp;
                if ((lane & 3) == 0) a.part_ml[cell] = make_float2(m_run[hf], l);
#pragma unroll
                for (int nt = 0; nt < HD / 8; nt++)
                    *reinterpret_cast<float2 *>(a.part_o + cell * HD + nt * 8 + (lane & 3) * 2) =
                        make_float2(o[nt][hf * 2], o[nt][hf * 2 + 1]);
            }
        }
    }
}

// Merge of the splits: one warp per (row, query head, 32 output dims).  Lane s holds split s's
// weight (att_splits <= 32); every lane owns one output dim and has all its loads in flight at once.
template <int HD>
__device__ __forceinline__ void mk_merge(const MkArgs &a)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    constexpr int PARTS = HD / 32;
    const int n_items = a.n_rows * a.Hq * PARTS;
    for (int item = warp * gridDim.x + blockIdx.x; item < n_items; item += gridDim.x * MK_CW) {
        const int cell = item / PARTS, d = (item % PARTS) * 32 + lane;
        const size_t cell0 = (size_t)cell * a.att_splits;
        float2 ml = make_float2(-INFINITY, 0.f);
        if (lane < a.att_splits) ml = a.part_ml[cell0 + lane];
        float v[MK_MAX_SPLITS];
#pragma unroll
        for (int s = 0; s < MK_MAX_SPLITS; s++) v[s] = s < a.att_splits ? a.part_o[(cell0 + s) * HD + d] : 0.f;
        const float M = warp_max(ml.x);
        const float w_mine = ml.x == -INFINITY ? 0.f : __expf(ml.x - M);
        const float den = warp_sum(ml.y * w_mine);
        float num = 0.f;
#pragma unroll
        for (int s = 0; s < MK_MAX_SPLITS; s++) num += v[s] * __shfl_sync(0xffffffffu, w_mine, s);
        a.attn_o[(size_t)cell * HD + d] = den > 0.f ? num / den : 0.f;
    }
}

}  // namespace sparsk

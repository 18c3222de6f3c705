// Attention and split-merge phases of the persistent layer-range kernel (see sparsk_mega.cuh).
#pragma once

namespace sparsk {

// Items (group, query block, kv head, split) are dealt to MK_ATT_WARPS warps of every CTA; a warp
// runs its item alone (attn_item of the stand-alone kernel): 16 query vectors (query heads of the
// kv head, for the group's rows) parked in shared memory (this kernel's register budget is spoken
// for), its own two-stage K/V ring inside the activation area, one partial per item.
template <int HD>
__device__ __forceinline__ void mk_attention(const MkArgs &a, const MkLayer *L, unsigned char *area, const MkShared *sh)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (warp >= MK_ATT_WARPS) return;
    // per warp: its 16 query vectors, then the K/V ring
    kv_t *qs = reinterpret_cast<kv_t *>(area) + (size_t)warp * (16 + MK_ATT_NST * 2 * AT_TP) * (HD + 8);
    kv_t *wr = qs + 16 * (HD + 8);
    AttnArgs at{};
    at.q = nullptr; at.q32 = a.q_buf; at.kc = L->kc; at.vc = L->vc;
    at.part_o = a.part_o; at.part_ml = a.part_ml;
    at.Hq = a.Hq; at.Hkv = a.Hkv; at.S = a.S; at.n_slots = a.n_slots; at.n_rows = a.n_rows;
    at.n_qblk = a.att_qblk; at.n_splits = a.att_splits; at.split_len = a.att_split_len; at.max_groups = a.n_groups;
    at.nq_min = 0; at.nq_max = 1 << 30;
    const unsigned n_workers = gridDim.x * MK_ATT_WARPS, worker = warp * gridDim.x + blockIdx.x;
    const unsigned n_items = (unsigned)a.n_groups * a.att_qblk * a.Hkv * a.att_splits;
    for (unsigned item = worker; item < n_items; item += n_workers) {
        const AtItem it = at_resolve(at, item, n_items, a.n_groups, sh->grp_row0, sh->grp_nrows, sh->row_slot, sh->row_pos);
        if (!it.valid) continue;
        // a single row's query heads (at most eight per kv head) take the transposed form
        if (it.nq <= 8) attn_item_t<HD, MK_ATT_NST, false>(at, it, wr, lane);
        else attn_item<HD, MK_ATT_NST, false>(at, it, wr, qs, lane);
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

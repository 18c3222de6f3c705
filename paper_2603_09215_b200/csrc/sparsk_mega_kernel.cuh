// The persistent layer-range kernel itself (see sparsk_mega.cuh).
#pragma once

namespace sparsk {

// Walks this CTA's ring items in consumption order: for every layer, for the four projection
// phases, for every segment the CTA owns, for every k-step.
struct MkCursor {
    int l, type, ks;
    MkWalk walk;
    MkSeg seg;
    uint32_t idx;
    bool done;

    __device__ void settle(const MkArgs &a)
    {
        // move to the next phase that has work for this CTA
        for (;;) {
            if (l >= a.layer_end) {
                done = true;
                return;
            }
            walk.init(type, a);
            if (walk.next(seg)) {
                ks = seg.ks0;
                return;
            }
            next_phase();
        }
    }
    __device__ void next_phase()
    {
        type = type == MK_QKV ? MK_OPROJ : (type == MK_OPROJ ? MK_GATEUP : (type == MK_GATEUP ? MK_DOWN : MK_QKV));
        if (type == MK_QKV) l++;
    }
    __device__ void init(const MkArgs &a)
    {
        l = a.layer_begin;
        type = MK_QKV;
        idx = 0;
        done = false;
        settle(a);
    }
    __device__ void advance(const MkArgs &a)
    {
        idx++;
        if (++ks < seg.ks1) return;
        if (walk.next(seg)) {
            ks = seg.ks0;
            return;
        }
        next_phase();
        settle(a);
    }
    __device__ int band() const { return seg.band; }
};

template <int M, int HD>
__global__ void __launch_bounds__(MK_THREADS, 1) mega_kernel(const MkArgs a)
{
    extern __shared__ __align__(1024) unsigned char mk_smem[];
    __shared__ MkShared sh;
    // the swizzled boxes of the tensor-core form need the ring on a 1024-byte boundary
    unsigned char *ring = mk_smem + ((1024u - (smem_u32(mk_smem) & 1023u)) & 1023u);  // MK_SLOTS x 16 KB
    unsigned char *area = ring + (size_t)MK_SLOTS * MK_SLOT_BYTES;     // activations / attention rings
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int s = 0; s < MK_SLOTS; s++) {
            mbar_init(&sh.full[s], 1);
            mbar_init(&sh.empty[s], MK_CW);
        }
        sh.giving_up = 0;
        sh.never = 0;
        for (int i = 0; i < MK_MAX_ROWS; i++) {
            sh.row_slot[i] = i < a.n_rows ? a.row_slot[i] : -1;
            sh.row_pos[i] = i < a.n_rows ? a.row_pos[i] : -1;
            sh.grp_row0[i] = i < a.n_groups ? a.grp_row0[i] : -1;
            sh.grp_nrows[i] = i < a.n_groups ? a.grp_nrows[i] : 0;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (warp >= MK_CW) {
        // ------------------------------------------------------------ producers
        const int p = warp - MK_CW;  // owns items p, p + 4, ... and with them ring slots p and p + 4
        MkCursor ld;
        ld.init(a);
        bool ok = true;
        while (!ld.done && ok) {
            if ((int)(ld.idx % MK_PW) == p) {
                const int s = ld.idx % MK_SLOTS;
                int go = 1;
                if (lane == 0) {
                    go = mbar_wait(&sh.empty[s], ((ld.idx / MK_SLOTS) & 1) ^ 1, &sh.giving_up, a.status) ? 1 : 0;
                    if (go) mbar_expect_tx(&sh.full[s], MK_SLOT_BYTES);
                }
                go = __shfl_sync(0xffffffffu, go, 0);
                if (!(ok = go != 0)) break;
                if (lane < 2) {
                    const CUtensorMap *map[2];
                    int row[2];
                    mk_band(ld.type, a, a.layers + ld.l, ld.band(), map, row);
                    const uint32_t dst = smem_u32(ring) + s * MK_SLOT_BYTES + lane * MK_BOX_BYTES;
                    if (M >= 3)  // the same box as four swizzled 64-column blocks (entries MKW_N on)
                        tma_load_3d(dst, map[lane] + MKW_N, &sh.full[s], 0, row[lane], ld.ks * (MK_BOX_COLS / 64));
                    else
                        tma_load_2d(dst, map[lane], &sh.full[s], ld.ks * MK_BOX_COLS, row[lane]);
                }
            }
            ld.advance(a);
        }
        // never leave with copies in flight: every slot this producer filled must have landed
        // (consumers that gave up no longer free slots, so wait on the full barriers, 2 ms each)
        if (lane == 0) {
            const uint32_t total = ld.idx;  // items before the point where this producer stopped
            for (int s = p; s < MK_SLOTS; s += MK_PW)
                if (total > (uint32_t)s) mbar_wait(&sh.full[s], ((total - 1 - s) / MK_SLOTS) & 1, &sh.never, nullptr, 2000000ull);
        }
    } else {
        // ------------------------------------------------------------ consumers
        uint32_t it = 0;
        unsigned long long epoch = a.bar_base;
        if (blockIdx.x == 0 && threadIdx.x == 0 && a.trace) a.trace[0] = global_ns();
        bool ok = true;
        const int qd = a.Hq * a.hd;
        for (int l = a.layer_begin; l < a.layer_end && ok; l++) {
            const MkLayer *L = a.layers + l;
            // q/k/v
            if (!(ok = mk_proj<M>(MK_QKV, a, L, area, a.d, a.h, nullptr, L->attn_gain, ring, &sh, it))) break;
            if (!(ok = mk_grid_barrier(a, &sh, epoch))) break;
            // attention and the merge of its splits
            mk_attention<HD>(a, L, area, &sh);
            if (!(ok = mk_grid_barrier(a, &sh, epoch))) break;
            mk_merge<HD>(a);
            if (!(ok = mk_grid_barrier(a, &sh, epoch))) break;
            // O-projection
            if (!(ok = mk_proj<M>(MK_OPROJ, a, L, area, qd, nullptr, a.attn_o, nullptr, ring, &sh, it))) break;
            if (!(ok = mk_grid_barrier(a, &sh, epoch))) break;
            // MLP
            if (!(ok = mk_proj<M>(MK_GATEUP, a, L, area, a.d, a.h, nullptr, L->mlp_gain, ring, &sh, it))) break;
            if (!(ok = mk_grid_barrier(a, &sh, epoch))) break;
            if (!(ok = mk_proj<M>(MK_DOWN, a, L, area, a.F, nullptr, a.act, nullptr, ring, &sh, it))) break;
            if (!(ok = mk_grid_barrier(a, &sh, epoch))) break;
        }
        if (!ok && threadIdx.x == 0) sh.giving_up = 1;
    }
    __syncthreads();
}

}  // namespace sparsk

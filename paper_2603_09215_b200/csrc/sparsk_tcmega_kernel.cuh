// The persistent tcgen05 layer kernel itself (see sparsk_tcmega.cuh).
#pragma once

namespace sparsk {

// A producer waits here until `need` grid barriers of this launch have been passed by every CTA,
// i.e. until the activations a GEMM phase reads are complete.
__device__ __forceinline__ bool tk_wait_epoch(const TkArgs &a, TkShared *sh, unsigned long long need)
{
    unsigned long long t0 = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (ld_acquire_u64(a.bar) >= need) return true;
        if ((spin & 63u) == 63u) {
            if (ld_volatile_i32(a.abort_word) || *(volatile int *)&sh->giving_up) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > GM_TIMEOUT_NS) {
                sh->giving_up = 1;
                atomicOr(a.status, ST_TIMEOUT);
                atomicExch(a.abort_word, 1);
                return false;
            }
        }
    }
}

// GEMM ending of one phase, by worker warps 0..3 (thread = weight row of an accumulator).
template <class Ending>
__device__ __forceinline__ bool tk_endings(const TkArgs &a, const TkGemm &g, const Ending &end, TkShared *sh,
                                           uint32_t &unit_it, int mma_n)
{
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    TileCtx tc;
    tc.row = warp * 32 + lane;
    tc.m0 = 0;
    tc.m_end = a.m_rows;
    tc.acc_stride = mma_n;
    tc.xchg = nullptr;
    const int acc_cols = 2 * mma_n;
    for (int u = blockIdx.x; u < g.n_units(); u += gridDim.x, unit_it++) {
        int kb0, kb1;
        tk_locate(g, u, tc.matrix, tc.unit_row, tc.split, kb0, kb1);
        const int buf = unit_it & 1;
        if (!mbar_wait(&sh->acc_full[buf], (unit_it >> 1) & 1, &sh->giving_up, a.status)) return false;
        tc_fence_after();
        tc.taddr = sh->tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * acc_cols);
        end.tile(tc);
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->acc_empty[buf]);
    }
    return true;
}

template <int HD>
__global__ void __launch_bounds__(TK_THREADS, 1) tcmega_kernel(const __grid_constant__ TkArgs a)
{
    extern __shared__ __align__(1024) unsigned char tk_smem[];
    __shared__ TkShared sh;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char *base = tk_smem + ((1024u - (smem_u32(tk_smem) & 1023u)) & 1023u);  // 1024-byte aligned
    const uint32_t ring = smem_u32(base);
    constexpr int SLOT = TK_A_BYTES + TK_B_BYTES;
    const int mma_n = (a.m_rows + 15) & ~15;
    const int b_tile = a.box_n * GM_BK * 2;
    const unsigned long long grid = gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TK_SLOTS; s++) {
            mbar_init(&sh.full_a[s], 1);
            mbar_init(&sh.full_b[s], 1);
            mbar_init(&sh.empty[s], 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(&sh.acc_full[b], 1);
            mbar_init(&sh.acc_empty[b], 4);
        }
        sh.giving_up = 0;
        sh.never = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == TK_WORKERS) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                     "r"(256)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp > TK_WORKERS) {
        // ------------------------------------------------------------ producers
        const int p = warp - TK_WORKERS - 1;
        uint32_t it = 0;
        bool ok = true;
        unsigned long long seen = a.bar_base;  // barrier count this warp has already observed
        for (int l = a.layer_begin; l < a.layer_end && ok; l++) {
            const TkLayer *L = a.layers + l;
            const int lr = l - a.layer_begin;
            for (int ph = TK_QKV; ph < TK_PHASES && ok; ph++) {
                if (!tk_is_gemm(ph)) continue;
                const TkGemm g = tk_gemm(ph, a);
                // activations: complete once every CTA has passed the barrier before this phase.
                // weights: the attention phase uses the ring's memory, so nothing may be copied
                // into it before the latest attention phase is over in this CTA (a CTA without
                // items in the phases in between would otherwise run ahead into it).
                const unsigned long long need_b = a.bar_base + grid * (unsigned long long)(lr * TK_PHASES + ph);
                const int att_done = ph > TK_ATTN ? lr * TK_PHASES + TK_ATTN + 1 : (lr > 0 ? (lr - 1) * TK_PHASES + TK_ATTN + 1 : 0);
                const unsigned long long need_a = a.bar_base + grid * (unsigned long long)att_done;
                const CUtensorMap *mb_hi = ph == TK_OPROJ ? &a.ao_hi : (ph == TK_DOWN ? &a.act_hi : &a.x_hi);
                const CUtensorMap *mb_lo = ph == TK_OPROJ ? &a.ao_lo : (ph == TK_DOWN ? &a.act_lo : &a.x_lo);
                for (int u = blockIdx.x; u < g.n_units() && ok; u += gridDim.x) {
                    int mat, unit_row, sp, kb0, kb1;
                    tk_locate(g, u, mat, unit_row, sp, kb0, kb1);
                    const CUtensorMap *ma = ph == TK_QKV ? (mat == 0 ? &L->wq : (mat == 1 ? &L->wk : &L->wv))
                                                         : (ph == TK_OPROJ ? &L->wo : (ph == TK_GATEUP ? &L->wg : &L->wd));
                    for (int kb = kb0; kb < kb1 && ok; kb++, it++) {
                        if ((int)(it % TK_PW) != p) continue;
                        const int s = it % TK_SLOTS;
                        const uint32_t st = ring + (uint32_t)s * SLOT;
                        int go = 1;
                        if (lane == 0) {
                            go = mbar_wait(&sh.empty[s], ((it / TK_SLOTS) & 1) ^ 1, &sh.giving_up, a.status) ? 1 : 0;
                            if (go && seen < need_a) go = tk_wait_epoch(a, &sh, need_a) ? 1 : 0;
                            if (go) mbar_expect_tx(&sh.full_a[s], TK_A_BYTES);
                        }
                        go = __shfl_sync(0xffffffffu, go, 0);
                        if (!(ok = go != 0)) break;
                        if (seen < need_a) seen = need_a;
                        if (lane == 0) tma_load_2d(st, ma, &sh.full_a[s], kb * GM_BK, unit_row);
                        if (lane == 1 && g.pair) tma_load_2d(st + GM_BLK_BYTES, &L->wu, &sh.full_a[s], kb * GM_BK, unit_row);
                        if (seen < need_b) {
                            if (lane == 0) go = tk_wait_epoch(a, &sh, need_b) ? 1 : 0;
                            go = __shfl_sync(0xffffffffu, go, 0);
                            if (!(ok = go != 0)) break;
                            seen = need_b;
                        }
                        // other CTAs wrote the activations with plain stores
                        asm volatile("fence.proxy.async;" ::: "memory");
                        if (lane == 0) mbar_expect_tx(&sh.full_b[s], (uint32_t)(2 * b_tile));
                        __syncwarp();
                        if (lane == 2) tma_load_2d(st + TK_A_BYTES, mb_hi, &sh.full_b[s], kb * GM_BK, 0);
                        if (lane == 3) tma_load_2d(st + TK_A_BYTES + b_tile, mb_lo, &sh.full_b[s], kb * GM_BK, 0);
                    }
                }
            }
        }
        // never leave with copies in flight
        if (lane == 0) {
            for (int s = p; s < TK_SLOTS; s += TK_PW)
                if (it > (uint32_t)s) {
                    const uint32_t par = ((it - 1 - s) / TK_SLOTS) & 1;
                    mbar_wait(&sh.full_a[s], par, &sh.never, nullptr, 2000000ull);
                    mbar_wait(&sh.full_b[s], par, &sh.never, nullptr, 2000000ull);
                }
        }
    } else if (warp == TK_WORKERS) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(mma_n);
            const int acc_cols = 2 * mma_n;
            uint32_t it = 0, unit_it = 0;
            bool ok = true;
            for (int l = a.layer_begin; l < a.layer_end && ok; l++) {
                for (int ph = TK_QKV; ph < TK_PHASES && ok; ph++) {
                    if (!tk_is_gemm(ph)) continue;
                    const TkGemm g = tk_gemm(ph, a);
                    const int acc1_off = GM_BLK_BYTES;  // accumulator 1's 128 weight rows follow accumulator 0's
                    for (int u = blockIdx.x; u < g.n_units() && ok; u += gridDim.x, unit_it++) {
                        int mat, unit_row, sp, kb0, kb1;
                        tk_locate(g, u, mat, unit_row, sp, kb0, kb1);
                        const int buf = unit_it & 1;
                        if (!(ok = mbar_wait(&sh.acc_empty[buf], ((unit_it >> 1) & 1) ^ 1, &sh.giving_up, a.status))) break;
                        tc_fence_after();
                        const uint32_t d0 = sh.tmem_base + (uint32_t)(buf * acc_cols);
                        int accum = 0;
                        for (int kb = kb0; kb < kb1; kb++, it++) {
                            const int s = it % TK_SLOTS;
                            const uint32_t par = (it / TK_SLOTS) & 1;
                            if (!(ok = mbar_wait(&sh.full_a[s], par, &sh.giving_up, a.status))) break;
                            if (!(ok = mbar_wait(&sh.full_b[s], par, &sh.giving_up, a.status))) break;
                            tc_fence_after();
                            const uint32_t a_addr = ring + (uint32_t)s * SLOT, b_addr = a_addr + TK_A_BYTES;
#pragma unroll
                            for (int kk = 0; kk < GM_BK / 16; kk++) {
                                const uint64_t db = umma_desc_sw128(b_addr + kk * 32);
                                const uint64_t dl = umma_desc_sw128(b_addr + b_tile + kk * 32);
                                const uint64_t da0 = umma_desc_sw128(a_addr + kk * 32);
                                const uint64_t da1 = umma_desc_sw128(a_addr + acc1_off + kk * 32);
                                umma_bf16(d0, da0, db, idesc, accum);
                                umma_bf16(d0, da0, dl, idesc, 1);
                                umma_bf16(d0 + mma_n, da1, db, idesc, accum);
                                umma_bf16(d0 + mma_n, da1, dl, idesc, 1);
                                accum = 1;
                            }
                            umma_commit(&sh.empty[s]);
                        }
                        if (ok) umma_commit(&sh.acc_full[buf]);
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------ workers
        unsigned long long epoch = a.bar_base;
        uint32_t unit_it = 0;
        if (blockIdx.x == 0 && threadIdx.x == 0 && a.trace) a.trace[0] = global_ns();
        bool ok = true;
        for (int l = a.layer_begin; l < a.layer_end && ok; l++) {
            const TkLayer *L = a.layers + l;
            for (int ph = 0; ph < TK_PHASES && ok; ph++) {
                switch (ph) {
                case TK_NORM_A: tk_norm(a, L->attn_gain, &sh); break;
                case TK_NORM_M: tk_norm(a, L->mlp_gain, &sh); break;
                case TK_FINISH: tk_qkv_finish(a, L); break;
                case TK_ATTN: tk_attention<HD>(a, L, base); break;
                case TK_MERGE: tk_merge<HD>(a); break;
                default:
                    if (warp < 4) {
                        const TkGemm g = tk_gemm(ph, a);
                        if (ph == TK_QKV) {
                            QkvEnd e;
                            e.q_out = a.q32; e.kc = L->kc; e.vc = L->vc; e.rope = a.rope; e.row_slot = a.row_slot;
                            e.row_pos = a.row_pos; e.partial = a.qkv_part; e.Hq = a.Hq; e.Hkv = a.Hkv; e.hd = a.hd; e.S = a.S;
                            ok = tk_endings(a, g, e, &sh, unit_it, mma_n);
                        } else if (ph == TK_GATEUP) {
                            GateUpEnd e;
                            e.u = a.act_hi_p; e.u_lo = a.act_lo_p; e.F = a.F;
                            ok = tk_endings(a, g, e, &sh, unit_it, mma_n);
                        } else {
                            ResidEnd e;
                            e.h = a.h; e.n_out = a.d; e.atomic = 1;
                            ok = tk_endings(a, g, e, &sh, unit_it, mma_n);
                        }
                        if (!ok) *(volatile int *)&sh.giving_up = 1;
                    }
                }
                if (!tk_grid_barrier(a, &sh, epoch)) ok = false;
                if (blockIdx.x == 0 && threadIdx.x == 0 && a.trace) a.trace[1 + (l - a.layer_begin) * TK_PHASES + ph] = global_ns();
            }
        }
    }
    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == TK_WORKERS) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(sh.tmem_base), "r"(256) : "memory");
    }
}

}  // namespace sparsk

// Split-KV attention for blocks of many query vectors on the 5th-generation tensor cores.
//
// A refresh step of a sequence with 16 query heads per kv head and three pending positions has
// 64 query vectors that share one K/V stream (Algorithm 1: the pending positions and the current
// one go through the upper layers as one causal block): 64 flop per cache byte and more for
// prefill chunks, where the warp-per-item mma.sync kernel of sparsk_attn.cuh would re-read the
// cache once per 16 query vectors.  This kernel runs the same arithmetic on tcgen05 (queries and
// softmax weights rounded to fp16 once, like the cache they multiply):
//
//   S = Q K^T : A = the block's query vectors (up to 128 rows, fp16) held in TMEM,
//               stored there once with tcgen05.st (lane = query vector, elements packed two per
//               column); B = a [64 positions x 128] K tile exactly as TMA delivers it from the
//               cache (K-major); accumulator [128 x 64] fp32 in TMEM
//   O += P V  : A = the tile's softmax weights (fp16), written by the softmax warps
//               straight into TMEM; B = the V tile as delivered (positions x head dim = MN-major);
//               accumulated over all tiles in a [128 x 128] fp32 TMEM accumulator that the softmax
//               warps rescale in place (tcgen05.ld / st) when a tile raises a row's reference maximum
// With both A operands in TMEM an MMA reads only its K or V slice from shared memory (2 or 4 KB
// instead of 6 or 8): with the operands in shared memory the MMAs ran at 80 and 120 cycles each
// against 32 and 64 at the tensor rate.  TMEM columns: scores 2 x 64, output 128, weights 2 x 32
// (of a 64-column slot each), queries 64 (of 128).
//
// CTA = (group, block of 128 query vectors, kv head, KV split); warp 0 issues the TMA copies of a
// K ring (TA_KST tiles) and a V ring (TA_VST tiles), warp 1 issues the MMAs and owns the TMEM
// allocation, warps 2..9 do the softmax (thread = query vector = TMEM lane, two warps per lane
// quadrant with half the columns each).  The scores and the weight planes are double buffered: a
// tile's scores and weights are formed while the product of the tile before it still runs.  The partials
// (unnormalised output, running max, running sum per split) have the layout of the other
// attention kernel, and attn_merge_kernel merges them.  Every wait is bounded.
#pragma once

#include "sparsk_attn.cuh"
#include "sparsk_gemm.cuh"

namespace sparsk {

constexpr int TA_THREADS = 320;   // TMA warp, MMA warp, eight softmax warps
constexpr int TA_QB = 128;      // query vectors per CTA (UMMA M)
constexpr int TA_NT = 64;       // positions per tile
constexpr int TA_HD = 128;      // head dimension this kernel is built for
constexpr int TA_KST = 4;        // K tiles in flight: tile t + 4 is requested when the scores of tile t are done
constexpr int TA_VST = 3;        // V tiles in flight: tile t + 3 is requested when the product of tile t is done
constexpr float TA_RAISE = 11.f;  // a row's reference maximum (in units of log2 e) moves only when a tile exceeds it by this much
constexpr int TA_T_BYTES = TA_NT * TA_HD * 2;        // one K or V tile: 16 KB
constexpr int TA_SMEM = 1024 + (TA_KST + TA_VST) * TA_T_BYTES;
// TMEM columns (all 512): scores 2 x 64, output 128, weights 2 x (hi 32 + lo 32), queries hi 64 + lo 64
constexpr int TA_C_S = 0, TA_C_O = 128, TA_C_P = 256, TA_C_Q = 384;

struct AttnTcArgs {
    AttnArgs a;        // q32, row and group arrays, partial buffers, shapes, the split plan
    int split_mult;    // this kernel's split s fills partial slot s * split_mult of the a.n_splits slots a
                       // row has (the slots in between are marked empty): its splits are split_mult times
                       // as long as those of the kernel that takes the small groups of the same launch set
    int *status;       // device status word (ST_TIMEOUT on a wait that ran out)
};

// MN-major operand with the 128-byte swizzle: 64 contiguous elements per row of 128 bytes, groups
// of eight rows 1024 bytes apart (stride offset), the next 64 elements `lbo` bytes on (leading offset).
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t smem_addr, uint32_t lbo_bytes)
{
    return (uint64_t)((smem_addr & 0x3ffffu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
           (1ull << 46) | (2ull << 61);
}
// fp16 x fp16 -> fp32 (the cache is fp16; operand format fields 0 = f16 where the weight GEMMs set
// 1 = bf16), M = 128, N = n, A K-major; B K-major or (b_mn) MN-major.
__device__ __forceinline__ uint32_t umma_idesc_f16_ex(int n, bool b_mn)
{
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(TA_QB >> 4) << 24) | (b_mn ? (1u << 16) : 0u);
}
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
          "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// D (+)= A B with the A operand in TMEM (lane = row, 16-bit elements packed two per column) and B in shared memory.
__device__ __forceinline__ void umma_f16_ts(uint32_t tmem_d, uint32_t tmem_a, uint64_t desc_b, uint32_t idesc, int accumulate)
{
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16])
{
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}

__global__ void __launch_bounds__(TA_THREADS, 1)
    attn_tc_kernel(const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v, const AttnTcArgs args)
{
    extern __shared__ __align__(1024) unsigned char ta_smem[];
    __shared__ __align__(8) uint64_t k_full[TA_KST], k_empty[TA_KST], v_full[TA_VST], v_empty[TA_VST], s_full[2], s_empty[2],
        p_full[2], o_full[2];
    __shared__ uint32_t tmem_base_s;
    __shared__ int giving_up_s, never_s;
    __shared__ float xch[3][2][TA_QB];  // [tile parity, or 2 for the final sums][column half][query vector]: what the two warps of a row exchange
    volatile int *giving_up = &giving_up_s;
    const AttnArgs &a = args.a;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t base = (smem_u32(ta_smem) + 1023u) & ~1023u;
    const uint32_t k0 = base, v0 = k0 + TA_KST * TA_T_BYTES;

    // ---- what this CTA works on (every thread computes the same); a CTA whose group belongs to
    // the other kernel, or does not exist, leaves before it sets anything up
    griddep_launch();
    griddep_wait();
    const int bx = blockIdx.x, hk = blockIdx.y, sp = blockIdx.z;
    const int g = bx / a.n_qblk, qb = bx % a.n_qblk;
    const int G = a.Hq / a.Hkv;
    bool live = g < *a.n_groups;
    int row0 = 0, nrows = 0;
    if (live) {
        row0 = a.grp_row0[g];
        nrows = a.grp_nrows[g];
        live = row0 >= 0 && nrows >= 1 && row0 + nrows <= a.n_rows;
    }
    const int nq = nrows * G, q0 = qb * TA_QB;
    live = live && q0 < nq && nq >= a.nq_min && nq <= a.nq_max;
    if (!live) return;
    const int nq_here = min(TA_QB, nq - q0);
    const int slot = a.row_slot[row0], pos0 = a.row_pos[row0];
    const bool sane = slot >= 0 && slot < a.n_slots && pos0 >= 0;
    const int last_row = (q0 + nq_here - 1) / G;
    const int kv_end_all = sane ? min(pos0 + last_row + 1, a.S) : 0;
    const int s_beg = sp * a.split_len;
    const int s_end = min(s_beg + a.split_len, kv_end_all);
    const int n_tiles = s_end > s_beg ? (s_end - s_beg + TA_NT - 1) / TA_NT : 0;
    const int cache_row0 = ((sane ? slot : 0) * a.Hkv + hk) * a.S;

    if (threadIdx.x == 0) {
        for (int s = 0; s < TA_KST; s++) {
            mbar_init(&k_full[s], 1);
            mbar_init(&k_empty[s], 1);
        }
        for (int s = 0; s < TA_VST; s++) {
            mbar_init(&v_full[s], 1);
            mbar_init(&v_empty[s], 1);
        }
        for (int b = 0; b < 2; b++) {
            mbar_init(&s_full[b], 1);
            mbar_init(&s_empty[b], 256);
            mbar_init(&p_full[b], 256);
            mbar_init(&o_full[b], 1);
        }
        giving_up_s = 0;
        never_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_s)), "r"(512)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }

    tc_fence_before();
    __syncthreads();  // the TMEM base address is known
    tc_fence_after();
    const uint32_t tmem_base = tmem_base_s;
    const uint32_t t_s0 = tmem_base + TA_C_S, t_o = tmem_base + TA_C_O, t_p = tmem_base + TA_C_P, t_q = tmem_base + TA_C_Q;

    // ---- the queries, as an fp16 plane in TMEM (thread = query vector = lane; 16-bit elements
    // packed two per column): the A operand of every score MMA, stored once.  The two warps of a
    // lane quadrant take 64 of the 128 head dimensions each.
    if (warp >= 2 && n_tiles > 0) {
        const int qi = (warp & 3) * 32 + lane, half = (warp - 2) >> 2;
        const bool have = qi < nq_here;
        const int qg = q0 + qi, r = qg / G, j = qg % G;
        const float *src = a.q32 + (size_t)(row0 + (have ? r : 0)) * a.Hq * TA_HD + (hk * G + (have ? j : 0)) * TA_HD + half * 64;
        const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
#pragma unroll
        for (int blk = 0; blk < 2; blk++) {  // 32 elements = 16 packed columns per store
            uint32_t hi[16];
#pragma unroll
            for (int c = 0; c < 4; c++) {
                uint4 h4 = make_uint4(0, 0, 0, 0);
                if (have) {
                    const float4 x0 = *reinterpret_cast<const float4 *>(src + blk * 32 + c * 8);
                    const float4 x1 = *reinterpret_cast<const float4 *>(src + blk * 32 + c * 8 + 4);
                    h4 = make_uint4(pack_h2(x0.x, x0.y), pack_h2(x0.z, x0.w), pack_h2(x1.x, x1.y), pack_h2(x1.z, x1.w));
                }
                hi[c * 4] = h4.x; hi[c * 4 + 1] = h4.y; hi[c * 4 + 2] = h4.z; hi[c * 4 + 3] = h4.w;
            }
            tmem_st16(t_q + lane_addr + (uint32_t)(half * 32 + blk * 16), hi);
        }
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    if (warp == 0) {
        // ------------------------------------------------------------ producer
        // One thread needs a few hundred nanoseconds per TMA copy, so a tile is two copies (the
        // [64][rows][2] view of the cache brings both 64-column halves of K, or of V, at once):
        // lane 0 runs the K ring, lane 1 the V ring, each at its own pace.
        if (lane < 2) {
            const bool is_v = lane == 1;
            const int depth = is_v ? TA_VST : TA_KST;
            uint64_t *full = is_v ? v_full : k_full, *empty = is_v ? v_empty : k_empty;
            const uint32_t ring0 = is_v ? v0 : k0;
            const CUtensorMap *map = is_v ? &map_v : &map_k;
            uint32_t issued = 0;
            for (int t = 0; t < n_tiles; t++) {
                const int st = t % depth;
                if (!mbar_wait(&empty[st], ((t / depth) & 1) ^ 1, giving_up, args.status)) break;
                mbar_expect_tx(&full[st], TA_T_BYTES);
                tma_load_3d(ring0 + (uint32_t)st * TA_T_BYTES, map, &full[st], 0, cache_row0 + s_beg + t * TA_NT, 0);
                issued++;
            }
            // never leave with copies in flight
            for (int st = 0; st < depth; st++)
                if (issued > (uint32_t)st)
                    mbar_wait(&full[st], ((issued - 1 - st) / depth) & 1, &never_s, nullptr, 2000000ull);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && n_tiles > 0) {
            const uint32_t idesc_s = umma_idesc_f16_ex(TA_NT, false), idesc_o = umma_idesc_f16_ex(TA_HD, true);
            bool ok = true;
            auto issue_s = [&](int t) {
                const int st = t % TA_KST, b = t & 1;
                if (!(ok = mbar_wait(&k_full[st], (t / TA_KST) & 1, giving_up, args.status))) return;
                if (!(ok = mbar_wait(&s_empty[b], ((t >> 1) & 1) ^ 1, giving_up, args.status))) return;
                tc_fence_after();
                // one thread issues every MMA, so the descriptors are built once and only advanced:
                // the address field (16-byte units, low 14 bits) takes the constant offsets by addition
                const uint64_t dk0 = umma_desc_sw128(k0 + (uint32_t)st * TA_T_BYTES);
                const uint32_t d = t_s0 + (uint32_t)b * TA_NT;
#pragma unroll
                for (int kk = 0; kk < TA_HD / 16; kk++) {  // 16 head dimensions = 8 packed TMEM columns of the queries
                    const uint64_t db = dk0 + (uint64_t)(((kk >> 2) * 8192 + (kk & 3) * 32) >> 4);
                    umma_f16_ts(d, t_q + (uint32_t)kk * 8, db, idesc_s, kk > 0);
                }
                umma_commit(&k_empty[st]);  // the K tile is free once the scores are computed
                umma_commit(&s_full[b]);
            };
            // order of issue: S(0), S(1), P.V(0), S(2), P.V(1), ...: a tile's scores never wait for
            // the weights of the tile before it
            issue_s(0);
            for (int t = 0; t < n_tiles && ok; t++) {
                if (t + 1 < n_tiles) issue_s(t + 1);
                if (!ok) break;
                const int st = t % TA_VST, b = t & 1;
                if (!(ok = mbar_wait(&v_full[st], (t / TA_VST) & 1, giving_up, args.status))) break;
                if (!(ok = mbar_wait(&p_full[b], (t >> 1) & 1, giving_up, args.status))) break;
                tc_fence_after();
                const uint64_t dv0 = umma_desc_sw128_mn(v0 + (uint32_t)st * TA_T_BYTES, 8192);
                const uint32_t tp = t_p + (uint32_t)b * 64;  // this tile's weights
#pragma unroll
                for (int kk = 0; kk < TA_NT / 16; kk++) {  // 16 positions = 8 packed columns
                    const uint64_t dv = dv0 + (uint64_t)((kk * 2048) >> 4);
                    umma_f16_ts(t_o, tp + (uint32_t)kk * 8, dv, idesc_o, t > 0 || kk > 0);
                }
                umma_commit(&v_empty[st]);  // the V tile and this buffer of weights are free once these have read them
                umma_commit(&o_full[b]);
            }
        }
    } else {
        // ------------------------------------------------------------ softmax and output (thread = query vector)
        // Two warps per TMEM lane quadrant: both own the same 32 query vectors (thread = query
        // vector), warp `half` takes score columns [32 half, 32 half + 32) and output columns
        // [64 half, 64 half + 64); they exchange their tile maxima (and at the end their sums)
        // through shared memory behind a 64-thread named barrier.
        const int quad = warp & 3, half = (warp - 2) >> 2, qi = quad * 32 + lane;
        const bool have = qi < nq_here;
        const int limit = have ? pos0 + (q0 + qi) / G : -1;
        const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
        const float scale = rsqrtf((float)TA_HD);
        float m_run = -INFINITY, l_run = 0.f;  // l_run: this warp's columns only
        bool ok = true;
        auto pair_sync = [&]() { asm volatile("bar.sync %0, 64;" ::"r"(8 + quad) : "memory"); };
        // The choice below is per quadrant: tcgen05.ld/st are warp-wide (.sync.aligned) instructions,
        // so a warp either runs the whole softmax path with all its lanes (lanes without a query
        // vector see everything masked) or none of it.
        const bool warp_idle = quad * 32 >= nq_here;
        if (warp_idle && n_tiles > 0) {
            // warps without query vectors: their rows of the weight planes stay zero, and they only
            // keep the barriers' arrival counts whole
            {   // both buffers, both planes, this warp's 16 columns of each
                uint32_t z[16];
#pragma unroll
                for (int i = 0; i < 16; i++) z[i] = 0u;
#pragma unroll
                for (int pl = 0; pl < 4; pl++) tmem_st16(t_p + lane_addr + (uint32_t)(pl * 32 + half * 16), z);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                tc_fence_before();
            }
            for (int t = 0; t < n_tiles && ok; t++) {
                if (!(ok = mbar_wait(&s_full[t & 1], (t >> 1) & 1, giving_up, args.status))) break;
                if (t >= 2 && !(ok = mbar_wait(&o_full[t & 1], ((t >> 1) - 1) & 1, giving_up, args.status))) break;
                mbar_arrive(&s_empty[t & 1]);
                mbar_arrive(&p_full[t & 1]);
            }
        } else if (n_tiles > 0) {
            // The output row accumulates in TMEM over all tiles (the MMAs add into it), relative to
            // the running maximum m_run; when a tile raises a row's maximum the warps rescale their
            // columns of the accumulator in place before the tile's product is issued.
            const float c2 = scale * 1.4426950408889634f;  // scores in units of log2(e)
            const int min_limit = __reduce_min_sync(0xffffffffu, have ? limit : 0x7fffffff);
            const bool all_have = __all_sync(0xffffffffu, have);
            for (int t = 0; t < n_tiles; t++) {
                const int b = t & 1;
                ok = ok && mbar_wait(&s_full[b], (t >> 1) & 1, giving_up, args.status);
                ok = __all_sync(0xffffffffu, ok);  // the loads below are warp-wide
                const uint32_t ts = t_s0 + lane_addr + (uint32_t)b * TA_NT + (uint32_t)half * 32;
                const int p0 = s_beg + t * TA_NT + half * 32;
                uint32_t sr[2][16];
                if (ok) {
                    tc_fence_after();
                    tmem_ld16_nowait(ts, sr[0]);
                    tmem_ld16_nowait(ts + 16, sr[1]);
                    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                    tc_fence_before();
                    mbar_arrive(&s_empty[b]);  // the scores are in registers
                } else {
#pragma unroll
                    for (int i = 0; i < 16; i++) sr[0][i] = sr[1][i] = 0xff800000u;  // -inf: keep going to the barriers below
                }
                // A tile that lies wholly inside what every row of the warp may see (the common case:
                // only a split's last tiles touch the causal edge or the split's end) needs no masking.
                const bool full_tile = p0 + 32 <= s_end && p0 + 31 <= min_limit && all_have;
                float tmax = -INFINITY;
                if (full_tile) {
#pragma unroll
                    for (int c = 0; c < 2; c++)
#pragma unroll
                        for (int i = 0; i < 16; i++) {
                            const float x = __uint_as_float(sr[c][i]) * c2;
                            sr[c][i] = __float_as_uint(x);
                            tmax = fmaxf(tmax, x);
                        }
                } else {
#pragma unroll
                    for (int c = 0; c < 2; c++)
#pragma unroll
                        for (int i = 0; i < 16; i++) {
                            const int p = p0 + c * 16 + i;
                            const float x = (p < s_end && p <= limit) ? __uint_as_float(sr[c][i]) * c2 : -INFINITY;
                            sr[c][i] = __float_as_uint(x);
                            tmax = fmaxf(tmax, x);
                        }
                }
                // the row's maximum over both halves (both warps always reach this barrier, also when giving up)
                xch[b][half][qi] = tmax;
                pair_sync();
                tmax = fmaxf(tmax, xch[b][half ^ 1][qi]);
                ok = ok && *giving_up == 0;
                if (!(ok = __all_sync(0xffffffffu, ok))) {
                    // leave together: the partner warp reads the same flag after the same barrier
                    break;
                }
                // The reference maximum is allowed to lag the true one by TA_RAISE (weights then reach
                // 2^11, which fp16 and fp32 sums carry at full precision): otherwise some lane of
                // the warp would see a new maximum in most tiles and the accumulator would be
                // rescaled nearly every time.  Partials stay exact: (o, l) are relative to m_run.
                const bool raise = tmax > m_run + TA_RAISE;
                const float m_new = raise ? tmax : m_run;
                const float factor = raise ? exp2f(m_run - m_new) : 1.f;  // 2^(-inf) = 0 on the first live tile
                const float m_ref = m_new == -INFINITY ? 0.f : m_new;    // a row that has seen nothing yet: all weights 0
                float psum = 0.f;
                uint4 whi[4];
#pragma unroll
                for (int c = 0; c < 4; c++) {
                    float w[8];
#pragma unroll
                    for (int i = 0; i < 8; i++) {
                        w[i] = exp2f(__uint_as_float(sr[c >> 1][(c & 1) * 8 + i]) - m_ref);  // 2^(-inf) = 0 for masked positions
                        psum += w[i];
                    }
                    whi[c] = make_uint4(pack_h2(w[0], w[1]), pack_h2(w[2], w[3]), pack_h2(w[4], w[5]), pack_h2(w[6], w[7]));
                }
                // The weights go to buffer b, which the product of tile t - 2 has read by the time
                // o_full[b] completes; a rescaling needs every product so far in the accumulator.  A
                // wait that fails here does not leave the loop on its own: the two warps of a row only
                // leave together, after the next named barrier (which has no time limit).
                if (t >= 2) {
                    ok = mbar_wait(&o_full[b], ((t >> 1) - 1) & 1, giving_up, args.status);
                    ok = __all_sync(0xffffffffu, ok);
                }
                if (ok && t > 0 && __any_sync(0xffffffffu, raise)) {
                    ok = mbar_wait(&o_full[(t - 1) & 1], ((t - 1) >> 1) & 1, giving_up, args.status);
                    ok = __all_sync(0xffffffffu, ok);
                    if (ok) {
                        tc_fence_after();
                        const uint32_t to = t_o + lane_addr + (uint32_t)half * 64;
#pragma unroll
                        for (int c0 = 0; c0 < 64; c0 += 32) {
                            uint32_t r0[16], r1[16];
                            tmem_ld16_nowait(to + c0, r0);
                            tmem_ld16_nowait(to + c0 + 16, r1);
                            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                            for (int i = 0; i < 16; i++) {
                                r0[i] = __float_as_uint(__uint_as_float(r0[i]) * factor);
                                r1[i] = __float_as_uint(__uint_as_float(r1[i]) * factor);
                            }
                            tmem_st16(to + c0, r0);
                            tmem_st16(to + c0 + 16, r1);
                        }
                        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    }
                }
                if (ok) {
                    uint32_t ph[16];
#pragma unroll
                    for (int c = 0; c < 4; c++) {
                        ph[c * 4] = whi[c].x; ph[c * 4 + 1] = whi[c].y; ph[c * 4 + 2] = whi[c].z; ph[c * 4 + 3] = whi[c].w;
                    }
                    const uint32_t tp = t_p + lane_addr + (uint32_t)(b * 64 + half * 16);
                    tmem_st16(tp, ph);
                    asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                    tc_fence_before();
                    mbar_arrive(&p_full[b]);
                }
                l_run = l_run * factor + psum;
                m_run = m_new;
            }
        }
        float o[64];
        if (!warp_idle && n_tiles > 0 && ok) {
            ok = mbar_wait(&o_full[(n_tiles - 1) & 1], ((n_tiles - 1) >> 1) & 1, giving_up, args.status);
            ok = __all_sync(0xffffffffu, ok);
            if (ok) {
                tc_fence_after();
                uint32_t r[4][16];
#pragma unroll
                for (int c = 0; c < 4; c++) tmem_ld16_nowait(t_o + lane_addr + (uint32_t)half * 64 + c * 16, r[c]);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int c = 0; c < 4; c++)
#pragma unroll
                    for (int i = 0; i < 16; i++) o[c * 16 + i] = __uint_as_float(r[c][i]);
                tc_fence_before();
            }
        } else {
#pragma unroll
            for (int i = 0; i < 64; i++) o[i] = 0.f;
        }
        // the row's sum over both halves (quadrants that ran the softmax path: both warps get here)
        if (!warp_idle && n_tiles > 0) {
            xch[2][half][qi] = l_run;
            pair_sync();
            l_run += xch[2][half ^ 1][qi];
        }
        if (have && ok) {
            const int qg = q0 + qi, r = qg / G, j = qg % G;
            const size_t cell0 = ((size_t)(row0 + r) * a.Hq + hk * G + j) * a.n_splits;
            const int first = sp * args.split_mult;
            if (first < a.n_splits) {
                float *dst = a.part_o + (cell0 + first) * TA_HD + half * 64;
#pragma unroll
                for (int i = 0; i < 64; i += 4) *reinterpret_cast<float4 *>(dst + i) = make_float4(o[i], o[i + 1], o[i + 2], o[i + 3]);
                if (half == 0) a.part_ml[cell0 + first] = make_float2(m_run * 0.6931471805599453f, l_run);  // back to natural-log units
            }
            if (half == 0)
                for (int e = first + 1; e < min(first + args.split_mult, a.n_splits); e++)
                    a.part_ml[cell0 + e] = make_float2(-INFINITY, 0.f);
        }
    }
    // ---------------------------------------------------------------- teardown
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
    }
}

}  // namespace sparsk

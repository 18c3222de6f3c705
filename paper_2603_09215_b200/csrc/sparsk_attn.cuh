// Split-KV grouped-query attention over the ragged KV cache (flash-decoding) on tensor cores.
//
// One CTA handles one (sequence group, block of query vectors, kv head, KV split).  A group is
// the block of rows of ONE sequence that a pass processes together: a single row in the lower
// pass, the pending positions plus the current one in the upper pass (Algorithm 1, full-depth
// branch: one causal block of at most K rows), a chunk of the prompt in prefill.  All query heads that share
// the kv head, for all rows of the group, form the M dimension of mma.sync m16n8k16 tiles, so one
// read of that head's K/V serves them all; row r of the group may look at positions
// <= pos0 + r (the causal mask of the block on top of the whole earlier cache).
//
// The split's positions are dealt to the CTA's four warps as contiguous sub-ranges.  Each warp
// streams its own 16-position K/V tiles into a private three-stage shared-memory ring with
// coalesced 16-byte cp.async copies (no CTA-wide barrier in the loop), computes S = Q K^T and
// O += P V with fp16 MMAs and fp32 accumulators (the cache is fp16; queries and softmax weights
// enter as two fp16 terms, hi + lo, so that only the cache itself is rounded), and keeps an online softmax whose row maxima
// and sums are reduced with shuffles inside the four-lane groups that share an accumulator row.
// The four warps' states are merged through shared memory into one unnormalised partial
// (acc, running max, running sum) per split; a second kernel merges the splits.
#pragma once

#include "sparsk_common.cuh"

namespace sparsk {

constexpr int AT_THREADS = 128;
constexpr int AT_TP = 16;        // positions per warp tile
constexpr int AT_NST = 3;        // ring stages per warp (two when the CTA holds 32 query vectors)
constexpr int AT_MAX_SPLITS = 32;
constexpr int AT_MIN_SPLIT = 64;

// How a launch cuts the work: query vectors per CTA (16 or 32), and the KV range into enough
// splits to fill the machine, none shorter than AT_MIN_SPLIT positions (unless forced), at most
// AT_MAX_SPLITS.
struct AttnPlan {
    int mt;  // m16 tiles per CTA: 1 or 2
    int n_qblk, split_len, n_splits;
};
inline AttnPlan attn_plan(int n_sm, int n_groups, int max_grp_rows, int G, int Hkv, int max_len, int forced_split)
{
    AttnPlan p;
    const int nq = max_grp_rows * G;
    p.mt = nq > 16 ? 2 : 1;
    p.n_qblk = (nq + 16 * p.mt - 1) / (16 * p.mt);
    int split = forced_split;
    if (split <= 0) {
        // Two CTAs fit an SM.  Cut the KV range so that the CTAs fill whole waves of 2 * n_sm and,
        // when the work allows, at least four of them (sequences are ragged and the causal cut
        // makes CTAs unequal: many short CTAs even that out); never below AT_MIN_SPLIT positions.
        const long slots = 2L * n_sm, base = (long)n_groups * p.n_qblk * Hkv;
        const int max_s = (int)(max_len / AT_MIN_SPLIT < 1 ? 1 : (max_len / AT_MIN_SPLIT > AT_MAX_SPLITS ? AT_MAX_SPLITS : max_len / AT_MIN_SPLIT));
        int best_s = 1;
        double best = -1.0;
        for (int s = 1; s <= max_s; s++) {
            const long n = base * s, waves = (n + slots - 1) / slots;
            const double eff = (double)n / (double)(waves * slots);
            if (waves >= 4 && eff >= 0.92) {
                best_s = s;
                break;
            }
            const double score = eff * (double)(waves < 4 ? waves : 4);
            if (score > best + 1e-9) {
                best = score;
                best_s = s;
            }
        }
        split = (max_len + best_s - 1) / best_s;
        if (split < AT_MIN_SPLIT) split = AT_MIN_SPLIT;
    }
    split = (split + AT_TP - 1) / AT_TP * AT_TP;
    int n_splits = (max_len + split - 1) / split;
    if (n_splits > AT_MAX_SPLITS) {
        n_splits = AT_MAX_SPLITS;
        split = ((max_len + n_splits - 1) / n_splits + AT_TP - 1) / AT_TP * AT_TP;
        n_splits = (max_len + split - 1) / split;
    }
    if (n_splits < 1) n_splits = 1;
    p.split_len = split;
    p.n_splits = n_splits;
    return p;
}
inline size_t attn_smem_bytes(int head_dim, int mt)
{
    const size_t kp = head_dim + 8;
    const size_t q = (size_t)2 * 16 * mt * kp * 2, ring = (size_t)4 * (mt == 2 ? 2 : AT_NST) * 2 * AT_TP * kp * 2;
    const size_t merge = (size_t)4 * 16 * mt * (head_dim + 2) * 4;
    return q + (ring > merge ? ring : merge);
}

struct AttnArgs {
    const bf16 *q;            // [rows][Hq*hd], already rotated
    const float *q32;         // the same in fp32; used instead of q when not NULL
    const kv_t *kc, *vc;      // this layer: [slot][Hkv][S][hd]
    const int *grp_row0, *grp_nrows, *row_slot, *row_pos;
    const int *n_groups;      // device count
    float *part_o;            // [rows*Hq][n_splits][hd]
    float2 *part_ml;          // [rows*Hq][n_splits]  (max, sum)
    bf16 *out;                // [rows][Hq*hd]
    bf16 *out_lo;             // optional second bf16 term: out + out_lo carries 16 significant bits
    int Hq, Hkv, S, n_qblk, n_splits, split_len;
    int n_slots;              // slots in the cache; rows naming another slot are skipped
    int n_rows;               // rows in q/out; groups reaching beyond them are skipped
    int nq_min, nq_max;       // only groups with this many query vectors per kv head (another launch takes the rest)
};

__device__ __forceinline__ void cp_async16(void *dst, const void *src, int src_bytes)
{
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src),
                 "r"(src_bytes)
                 : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait()
{
    asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t (&r)[4], const void *p)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t (&r)[4], const void *p)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"((uint32_t)__cvta_generic_to_shared(p)));
}
// D += A B, A 16x16 fp16 (row), B 16x8 fp16 (col), D 16x8 fp32.
__device__ __forceinline__ void mma_f16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// The work of one CTA (group * n_qblk + query block, kv head, split) by 128 threads; `sync` is the
// barrier of those threads.  Also the attention phase of the persistent layer kernel, which runs
// it on four-warp groups over virtual block indices.
struct AttnCtaSync {
    __device__ void operator()() const { __syncthreads(); }
};
template <int HD, int MT, int NS, class Sync>
__device__ __forceinline__ void attn_partial_body(const AttnArgs &a, int bx, int hk, int sp, unsigned char *at_smem, int tid,
                                                  Sync sync)
{
    constexpr int QB = 16 * MT;     // query vectors per CTA
    constexpr int KP = HD + 8;      // padded row: ldmatrix rows fall into distinct banks
    constexpr int CH = HD / 8;      // 16-byte chunks per row
    kv_t *Qs = reinterpret_cast<kv_t *>(at_smem);  // [QB][KP] hi terms
    kv_t *Ql = Qs + QB * KP;                       // [QB][KP] lo terms
    kv_t *ring = Ql + QB * KP;                     // [4 warps][NS][K,V][AT_TP][KP]

    const int g = bx / a.n_qblk, qb = bx % a.n_qblk;
    if (g >= *a.n_groups) return;
    const int G = a.Hq / a.Hkv;
    const int row0 = a.grp_row0[g], nrows = a.grp_nrows[g];
    if (row0 < 0 || nrows < 1 || row0 + nrows > a.n_rows) return;
    const int nq = nrows * G;
    const int q0 = qb * QB;
    if (q0 >= nq || nq < a.nq_min || nq > a.nq_max) return;
    const int nq_here = min(QB, nq - q0);
    const int slot = a.row_slot[row0], pos0 = a.row_pos[row0];
    const int lane = tid & 31, warp = tid >> 5;

    // positions this CTA may look at: its split, cut at the last query row's own position
    // (and at the cache itself: a descriptor that points outside it reads nothing)
    const int last_row = (q0 + nq_here - 1) / G;
    const bool sane = slot >= 0 && slot < a.n_slots && pos0 >= 0;
    const int kv_end_all = sane ? min(pos0 + last_row + 1, a.S) : 0;
    const int s_beg = sp * a.split_len;
    const int s_end = min(s_beg + a.split_len, kv_end_all);

    for (int i = tid; i < QB * CH; i += AT_THREADS) {
        const int qi = i / CH, c = i % CH;
        uint4 hi = make_uint4(0, 0, 0, 0), lo = hi;
        if (qi < nq_here) {
            const int qg = q0 + qi, r = qg / G, j = qg % G;
            const size_t off = (size_t)(row0 + r) * a.Hq * HD + (hk * G + j) * HD + c * 8;
            if (a.q32) {
                const float4 x0 = *reinterpret_cast<const float4 *>(a.q32 + off);
                const float4 x1 = *reinterpret_cast<const float4 *>(a.q32 + off + 4);
                const float v[8] = {x0.x, x0.y, x0.z, x0.w, x1.x, x1.y, x1.z, x1.w};
                split8_h(v, hi, lo);
            } else {
                float v[8];
                unpack8(*reinterpret_cast<const uint4 *>(a.q + off), v);  // bf16 queries, widened
                split8_h(v, hi, lo);
            }
        }
        *reinterpret_cast<uint4 *>(&Qs[qi * KP + c * 8]) = hi;
        *reinterpret_cast<uint4 *>(&Ql[qi * KP + c * 8]) = lo;
    }
    sync();

    // this warp's share of the split
    const int span = max(s_end - s_beg, 0);
    const int per = (((span + 3) >> 2) + AT_TP - 1) / AT_TP * AT_TP;
    const int w_beg = s_beg + warp * per;
    const int w_end = min(w_beg + per, s_end);
    const int n_tiles = w_end > w_beg ? (w_end - w_beg + AT_TP - 1) / AT_TP : 0;
    kv_t *wr = ring + (size_t)warp * NS * 2 * AT_TP * KP;
    const kv_t *kbase = a.kc + ((size_t)(sane ? slot : 0) * a.Hkv + hk) * a.S * HD;
    const kv_t *vbase = a.vc + ((size_t)(sane ? slot : 0) * a.Hkv + hk) * a.S * HD;

    auto issue = [&](int t) {
        kv_t *kt = wr + (size_t)(t % NS) * 2 * AT_TP * KP, *vt = kt + AT_TP * KP;
        const int p0 = w_beg + t * AT_TP;
#pragma unroll
        for (int i = lane; i < AT_TP * CH; i += 32) {
            const int r = i / CH, c = i % CH;
            const bool ok = p0 + r < w_end;                  // rows past the end are zero-filled
            const size_t off = (size_t)(ok ? p0 + r : w_beg) * HD + c * 8;
            cp_async16(&kt[r * KP + c * 8], kbase + off, ok ? 16 : 0);
            cp_async16(&vt[r * KP + c * 8], vbase + off, ok ? 16 : 0);
        }
    };

    float o[MT][HD / 8][4], m_run[MT][2], l_run[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; mt++) {
        m_run[mt][0] = m_run[mt][1] = -INFINITY;
        l_run[mt][0] = l_run[mt][1] = 0.f;
#pragma unroll
        for (int nt = 0; nt < HD / 8; nt++)
#pragma unroll
            for (int e = 0; e < 4; e++) o[mt][nt][e] = 0.f;
    }
    // last position each of this thread's accumulator rows may see
    int limit[MT][2];
#pragma unroll
    for (int mt = 0; mt < MT; mt++)
#pragma unroll
        for (int hf = 0; hf < 2; hf++) {
            const int qi = mt * 16 + (lane >> 2) + hf * 8;
            limit[mt][hf] = qi < nq_here ? pos0 + (q0 + qi) / G : -1;
        }
    const float scale = rsqrtf((float)HD);

#pragma unroll
    for (int t = 0; t < NS - 1; t++) {
        if (t < n_tiles) issue(t);
        cp_async_commit();
    }
    for (int t = 0; t < n_tiles; t++) {
        cp_async_wait<NS - 2>();
        __syncwarp();
        if (t + NS - 1 < n_tiles) issue(t + NS - 1);
        cp_async_commit();
        const kv_t *Kt = wr + (size_t)(t % NS) * 2 * AT_TP * KP, *Vt = Kt + AT_TP * KP;
        const int p0 = w_beg + t * AT_TP;

        // S = Q K^T for 16 positions
        float s[MT][2][4];
#pragma unroll
        for (int mt = 0; mt < MT; mt++)
#pragma unroll
            for (int nt = 0; nt < 2; nt++)
#pragma unroll
                for (int e = 0; e < 4; e++) s[mt][nt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ks++) {
            uint32_t kb[4];
            ldsm_x4(kb, &Kt[((lane & 7) + ((lane >> 4) << 3)) * KP + ks * 16 + ((lane >> 3) & 1) * 8]);
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {
                uint32_t qa[4], ql[4];
                const int qoff = (mt * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * KP + ks * 16 + (lane >> 4) * 8;
                ldsm_x4(qa, &Qs[qoff]);
                ldsm_x4(ql, &Ql[qoff]);
                mma_f16(s[mt][0], qa, kb[0], kb[1]);
                mma_f16(s[mt][1], qa, kb[2], kb[3]);
                mma_f16(s[mt][0], ql, kb[0], kb[1]);
                mma_f16(s[mt][1], ql, kb[2], kb[3]);
            }
        }
        // online softmax; P as the A operand of the second product
        uint32_t pa[MT][4], pl[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; mt++) {
#pragma unroll
            for (int hf = 0; hf < 2; hf++) {
                float v[4];
                float tmax = -INFINITY;
#pragma unroll
                for (int nt = 0; nt < 2; nt++)
#pragma unroll
                    for (int e = 0; e < 2; e++) {
                        const int p = p0 + nt * 8 + (lane & 3) * 2 + e;
                        const bool ok = p < w_end && p <= limit[mt][hf];
                        v[nt * 2 + e] = ok ? s[mt][nt][hf * 2 + e] * scale : -INFINITY;
                        tmax = fmaxf(tmax, v[nt * 2 + e]);
                    }
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
                tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
                const float m_new = fmaxf(m_run[mt][hf], tmax);
                float alpha = 1.f, psum = 0.f;
                if (m_new != -INFINITY) {
                    alpha = __expf(m_run[mt][hf] - m_new);  // exp(-inf) = 0 on the first live tile
#pragma unroll
                    for (int i = 0; i < 4; i++) {
                        v[i] = __expf(v[i] - m_new);
                        psum += v[i];
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < 4; i++) v[i] = 0.f;
                }
                l_run[mt][hf] = l_run[mt][hf] * alpha + psum;  // per-thread share; lanes are summed at the end
                m_run[mt][hf] = m_new;
                split_pair_h(v[0], v[1], pa[mt][hf], pl[mt][hf]);          // positions 0..7 of the tile
                split_pair_h(v[2], v[3], pa[mt][2 + hf], pl[mt][2 + hf]);  // positions 8..15
#pragma unroll
                for (int nt = 0; nt < HD / 8; nt++) {
                    o[mt][nt][hf * 2] *= alpha;
                    o[mt][nt][hf * 2 + 1] *= alpha;
                }
            }
        }
        // O += P V
#pragma unroll
        for (int np = 0; np < HD / 16; np++) {
            uint32_t vb[4];
            ldsm_x4_t(vb, &Vt[((lane & 7) + ((lane >> 3) & 1) * 8) * KP + np * 16 + (lane >> 4) * 8]);
#pragma unroll
            for (int mt = 0; mt < MT; mt++) {
                mma_f16(o[mt][2 * np], pa[mt], vb[0], vb[1]);
                mma_f16(o[mt][2 * np + 1], pa[mt], vb[2], vb[3]);
                mma_f16(o[mt][2 * np], pl[mt], vb[0], vb[1]);
                mma_f16(o[mt][2 * np + 1], pl[mt], vb[2], vb[3]);
            }
        }
    }
    cp_async_wait<0>();
    sync();  // every warp is done with its ring: reuse it for the merge

    // merge the four warps' states
    float *Ow = reinterpret_cast<float *>(ring);   // [4][QB][HD]
    float *mw = Ow + 4 * QB * HD, *lw = mw + 4 * QB;  // [4][QB] each
#pragma unroll
    for (int mt = 0; mt < MT; mt++)
#pragma unroll
        for (int hf = 0; hf < 2; hf++) {
            float l = l_run[mt][hf];
            l += __shfl_xor_sync(0xffffffffu, l, 1);
            l += __shfl_xor_sync(0xffffffffu, l, 2);
            const int qi = mt * 16 + (lane >> 2) + hf * 8;
            if ((lane & 3) == 0) {
                mw[warp * QB + qi] = m_run[mt][hf];
                lw[warp * QB + qi] = l;
            }
#pragma unroll
            for (int nt = 0; nt < HD / 8; nt++) {
                float2 v2 = make_float2(o[mt][nt][hf * 2], o[mt][nt][hf * 2 + 1]);
                *reinterpret_cast<float2 *>(&Ow[((size_t)warp * QB + qi) * HD + nt * 8 + (lane & 3) * 2]) = v2;
            }
        }
    sync();
    // partials (an empty split leaves max = -inf, sum = 0, which the merge of the splits ignores)
    for (int idx = tid; idx < nq_here * HD; idx += AT_THREADS) {
        const int qi = idx / HD, d = idx % HD;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; w++) M = fmaxf(M, mw[w * QB + qi]);
        float acc = 0.f, L = 0.f;
#pragma unroll
        for (int w = 0; w < 4; w++) {
            const float mwv = mw[w * QB + qi];
            if (mwv == -INFINITY) continue;
            const float wgt = __expf(mwv - M);
            acc += Ow[((size_t)w * QB + qi) * HD + d] * wgt;
            L += lw[w * QB + qi] * wgt;
        }
        const int qg = q0 + qi, r = qg / G, j = qg % G;
        const size_t cell = ((size_t)(row0 + r) * a.Hq + hk * G + j) * a.n_splits + sp;
        a.part_o[cell * HD + d] = acc;
        if (d == 0) a.part_ml[cell] = make_float2(M, L);
    }
}

template <int HD, int MT>
__global__ void __launch_bounds__(AT_THREADS) attn_partial_kernel(AttnArgs a)
{
    extern __shared__ __align__(16) unsigned char at_smem_dyn[];
    griddep_launch();
    griddep_wait();
    attn_partial_body<HD, MT, (MT == 2 ? 2 : AT_NST)>(a, blockIdx.x, blockIdx.y, blockIdx.z, at_smem_dyn, threadIdx.x,
                                                      AttnCtaSync());
}

typedef void (*AttnPartialFn)(AttnArgs);
// The instantiation for a head dimension (64 or 128) and a query block of 16 * mt vectors, with
// its dynamic shared-memory limit raised on first use.
inline cudaError_t attn_partial_fn(int head_dim, int mt, AttnPartialFn *fn)
{
    static PerDevice<bool> ready_dev[4];
    const int idx = (head_dim == 128 ? 2 : 0) + (mt == 2 ? 1 : 0);
    AttnPartialFn f = idx == 3 ? attn_partial_kernel<128, 2>
                      : idx == 2 ? attn_partial_kernel<128, 1>
                      : idx == 1 ? attn_partial_kernel<64, 2>
                                 : attn_partial_kernel<64, 1>;
    bool &ready = ready_dev[idx].here();
    if (!ready) {
        const cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)attn_smem_bytes(head_dim, mt));
        if (e != cudaSuccess) return e;
        ready = true;
    }
    *fn = f;
    return cudaSuccess;
}

// Merge the splits of every (row, query head): out = sum_s acc_s e^{m_s - M} / sum_s l_s e^{m_s - M}.
template <int HD>
__global__ void __launch_bounds__(HD) attn_merge_kernel(AttnArgs a, const int *__restrict__ n_rows)
{
    griddep_launch();
    griddep_wait();
    const int row = blockIdx.x, head = blockIdx.y;
    if (row >= *n_rows) return;
    const size_t cell0 = ((size_t)row * a.Hq + head) * a.n_splits;
    float M = -INFINITY;
    for (int s = 0; s < a.n_splits; s++) M = fmaxf(M, a.part_ml[cell0 + s].x);
    float den = 0.f, num = 0.f;
    for (int s = 0; s < a.n_splits; s++) {
        const float2 ml = a.part_ml[cell0 + s];
        if (ml.x == -INFINITY) continue;
        const float w = __expf(ml.x - M);
        den += ml.y * w;
        num += a.part_o[(cell0 + s) * HD + threadIdx.x] * w;
    }
    const float val = den > 0.f ? num / den : 0.f;
    const bf16 hi = __float2bfloat16(val);
    a.out[(size_t)row * a.Hq * HD + head * HD + threadIdx.x] = hi;
    if (a.out_lo) a.out_lo[(size_t)row * a.Hq * HD + head * HD + threadIdx.x] = __float2bfloat16(val - __bfloat162float(hi));
}

}  // namespace sparsk

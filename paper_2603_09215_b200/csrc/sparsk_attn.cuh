// Split-KV grouped-query attention over the ragged KV cache (flash-decoding).
//
// One CTA handles one (sequence group, block of query vectors, kv head, KV split).  A group is
// the block of rows of ONE sequence that a pass processes together: a single row in the lower
// pass, the pending positions plus the current one in the upper pass (Algorithm 1: "batch
// P u {t} ... length-K mask"), a chunk of the prompt in prefill.  All query heads that share
// the kv head, for all rows of the group, are served from one read of that head's K/V tile;
// row r of the group may look at positions <= pos0 + r (the causal mask of the block on top
// of the whole earlier cache).  K/V tiles are fetched with coalesced 16-byte loads; softmax
// statistics are reduced with warp shuffles; each split writes an unnormalised partial
// (acc, running max, running sum) and a second kernel merges the splits.
#pragma once

#include "sparsk_common.cuh"

namespace sparsk {

constexpr int AT_THREADS = 128;
constexpr int AT_QB = 32;    // query vectors per CTA
constexpr int AT_TILE = 32;  // KV positions per tile
constexpr int AT_MAX_SPLITS = 32;
constexpr int AT_MIN_SPLIT = 64;

// How a launch cuts the KV range: enough splits to fill the machine, none shorter than
// AT_MIN_SPLIT positions (unless forced), at most AT_MAX_SPLITS.
struct AttnPlan {
    int n_qblk, split_len, n_splits;
};
inline AttnPlan attn_plan(int n_sm, int n_groups, int max_grp_rows, int G, int Hkv, int max_len, int forced_split)
{
    AttnPlan p;
    p.n_qblk = (max_grp_rows * G + AT_QB - 1) / AT_QB;
    int split = forced_split;
    if (split <= 0) {
        const long base = (long)n_groups * p.n_qblk * Hkv;
        long want = (2L * n_sm + base - 1) / base;
        want = want < 1 ? 1 : (want > AT_MAX_SPLITS ? AT_MAX_SPLITS : want);
        split = (int)((max_len + want - 1) / want);
        if (split < AT_MIN_SPLIT) split = AT_MIN_SPLIT;
    }
    split = (split + AT_TILE - 1) / AT_TILE * AT_TILE;
    int n_splits = (max_len + split - 1) / split;
    if (n_splits > AT_MAX_SPLITS) {
        n_splits = AT_MAX_SPLITS;
        split = ((max_len + n_splits - 1) / n_splits + AT_TILE - 1) / AT_TILE * AT_TILE;
        n_splits = (max_len + split - 1) / split;
    }
    if (n_splits < 1) n_splits = 1;
    p.split_len = split;
    p.n_splits = n_splits;
    return p;
}

struct AttnArgs {
    const bf16 *q;            // [rows][Hq*hd], already rotated
    const bf16 *kc, *vc;      // this layer: [slot][Hkv][S][hd]
    const int *grp_row0, *grp_nrows, *row_slot, *row_pos;
    const int *n_groups;      // device count
    float *part_o;            // [rows*Hq][n_splits][hd]
    float2 *part_ml;          // [rows*Hq][n_splits]  (max, sum)
    bf16 *out;                // [rows][Hq*hd]
    int Hq, Hkv, S, n_qblk, n_splits, split_len;
    int n_slots;              // slots in the cache; rows naming another slot are skipped
    int n_rows;               // rows in q/out; groups reaching beyond them are skipped
};

template <int HD>
__global__ void __launch_bounds__(AT_THREADS) attn_partial_kernel(AttnArgs a)
{
    constexpr int KP = HD + 8;  // padded row, keeps 16-byte row reads conflict-free
    __shared__ __align__(16) float qs[AT_QB][HD];
    __shared__ __align__(16) bf16 Ks[AT_TILE][KP];
    __shared__ __align__(16) bf16 Vs[AT_TILE][KP];
    __shared__ float Ps[AT_QB][AT_TILE];

    griddep_wait();
    griddep_launch();
    const int g = blockIdx.x / a.n_qblk, qb = blockIdx.x % a.n_qblk;
    if (g >= *a.n_groups) return;
    const int hk = blockIdx.y, sp = blockIdx.z;
    const int G = a.Hq / a.Hkv;
    const int row0 = a.grp_row0[g], nrows = a.grp_nrows[g];
    if (row0 < 0 || nrows < 1 || row0 + nrows > a.n_rows) return;
    const int nq = nrows * G;
    const int q0 = qb * AT_QB;
    if (q0 >= nq) return;
    const int nq_here = min(AT_QB, nq - q0);
    const int slot = a.row_slot[row0], pos0 = a.row_pos[row0];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // positions this CTA may look at: its split, cut at the last query row's own position
    // (and at the cache itself: a descriptor that points outside it reads nothing)
    const int last_row = (q0 + nq_here - 1) / G;
    const bool sane = slot >= 0 && slot < a.n_slots && pos0 >= 0;
    const int kv_end_all = sane ? min(pos0 + last_row + 1, a.S) : 0;
    const int s_beg = sp * a.split_len;
    const int s_end = min(s_beg + a.split_len, kv_end_all);

    // queries -> shared, pre-scaled by 1/sqrt(hd)
    const float scale = rsqrtf((float)HD);
    for (int i = tid; i < AT_QB * (HD / 8); i += AT_THREADS) {
        const int qi = i / (HD / 8), c = i % (HD / 8);
        float f[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        if (qi < nq_here) {
            const int qg = q0 + qi, r = qg / G, j = qg % G;
            unpack8(*reinterpret_cast<const uint4 *>(a.q + (size_t)(row0 + r) * a.Hq * HD + (hk * G + j) * HD + c * 8), f);
        }
#pragma unroll
        for (int e = 0; e < 8; e++) qs[qi][c * 8 + e] = f[e] * scale;
    }

    constexpr int QW = AT_QB / 4;   // query vectors per warp
    constexpr int DL = HD / 32;     // output dims per lane
    float m_run[QW], l_run[QW], acc[QW][DL];
#pragma unroll
    for (int i = 0; i < QW; i++) {
        m_run[i] = -INFINITY;
        l_run[i] = 0.f;
#pragma unroll
        for (int e = 0; e < DL; e++) acc[i][e] = 0.f;
    }
    const bf16 *kbase = a.kc + ((size_t)slot * a.Hkv + hk) * a.S * HD;
    const bf16 *vbase = a.vc + ((size_t)slot * a.Hkv + hk) * a.S * HD;

    for (int t0 = s_beg; t0 < s_end; t0 += AT_TILE) {
        __syncthreads();  // previous tile fully consumed (also orders the query stores)
        for (int i = tid; i < AT_TILE * (HD / 8); i += AT_THREADS) {
            const int t = i / (HD / 8), c = i % (HD / 8);
            uint4 kv = make_uint4(0, 0, 0, 0), vv = make_uint4(0, 0, 0, 0);
            if (t0 + t < s_end) {
                kv = ld_stream16(kbase + (size_t)(t0 + t) * HD + c * 8);
                vv = ld_stream16(vbase + (size_t)(t0 + t) * HD + c * 8);
            }
            *reinterpret_cast<uint4 *>(&Ks[t][c * 8]) = kv;
            *reinterpret_cast<uint4 *>(&Vs[t][c * 8]) = vv;
        }
        __syncthreads();
        // scores: lane = position, each warp walks its QW query vectors
        const int tpos = t0 + lane;
        float sc[QW];
#pragma unroll
        for (int i = 0; i < QW; i++) sc[i] = 0.f;
#pragma unroll 4
        for (int c = 0; c < HD / 8; c++) {
            float kf[8];
            unpack8(*reinterpret_cast<const uint4 *>(&Ks[lane][c * 8]), kf);
#pragma unroll
            for (int i = 0; i < QW; i++) {
                const float4 qa = *reinterpret_cast<const float4 *>(&qs[warp * QW + i][c * 8]);
                const float4 qb4 = *reinterpret_cast<const float4 *>(&qs[warp * QW + i][c * 8 + 4]);
                sc[i] += kf[0] * qa.x + kf[1] * qa.y + kf[2] * qa.z + kf[3] * qa.w + kf[4] * qb4.x +
                         kf[5] * qb4.y + kf[6] * qb4.z + kf[7] * qb4.w;
            }
        }
#pragma unroll
        for (int i = 0; i < QW; i++) {
            const int qi = warp * QW + i;
            const int r = (q0 + qi) / G;
            const bool ok = qi < nq_here && tpos < s_end && tpos <= pos0 + r;
            const float s = ok ? sc[i] : -INFINITY;
            const float m_new = fmaxf(m_run[i], warp_max(s));
            float alpha = 1.f, p = 0.f;
            if (m_new != -INFINITY) {
                alpha = __expf(m_run[i] - m_new);  // exp(-inf) = 0 on the first live tile
                p = __expf(s - m_new);
            }
            l_run[i] = l_run[i] * alpha + warp_sum(p);
            m_run[i] = m_new;
            Ps[qi][lane] = p;
#pragma unroll
            for (int e = 0; e < DL; e++) acc[i][e] *= alpha;
        }
        __syncwarp();
        // acc += P V : lane owns DL consecutive output dims
        for (int t = 0; t < AT_TILE; t++) {
            float vf[DL];
            if constexpr (DL == 4) {
                const uint2 v2 = *reinterpret_cast<const uint2 *>(&Vs[t][lane * 4]);
                vf[0] = bf_lo(v2.x); vf[1] = bf_hi(v2.x); vf[2] = bf_lo(v2.y); vf[3] = bf_hi(v2.y);
            } else {
                const uint32_t v1 = *reinterpret_cast<const uint32_t *>(&Vs[t][lane * 2]);
                vf[0] = bf_lo(v1); vf[1] = bf_hi(v1);
            }
#pragma unroll
            for (int i = 0; i < QW; i++) {
                const float p = Ps[warp * QW + i][t];
#pragma unroll
                for (int e = 0; e < DL; e++) acc[i][e] = fmaf(p, vf[e], acc[i][e]);
            }
        }
    }
    // partials (an empty split leaves max = -inf, sum = 0, which the merge ignores)
#pragma unroll
    for (int i = 0; i < QW; i++) {
        const int qi = warp * QW + i;
        if (qi >= nq_here) continue;
        const int qg = q0 + qi, r = qg / G, j = qg % G;
        const size_t cell = ((size_t)(row0 + r) * a.Hq + hk * G + j) * a.n_splits + sp;
        float *po = a.part_o + cell * HD + lane * DL;
#pragma unroll
        for (int e = 0; e < DL; e++) po[e] = acc[i][e];
        if (lane == 0) a.part_ml[cell] = make_float2(m_run[i], l_run[i]);
    }
}

// Merge the splits of every (row, query head): out = sum_s acc_s e^{m_s - M} / sum_s l_s e^{m_s - M}.
template <int HD>
__global__ void __launch_bounds__(HD) attn_merge_kernel(AttnArgs a, const int *__restrict__ n_rows)
{
    griddep_wait();
    griddep_launch();
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
    a.out[(size_t)row * a.Hq * HD + head * HD + threadIdx.x] = __float2bfloat16(den > 0.f ? num / den : 0.f);
}

}  // namespace sparsk

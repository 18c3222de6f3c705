// Small-batch weight-streaming path: y = W x for up to four activation rows at a time.
//
// At a handful of rows a transformer layer is bound by reading its weights from HBM once
// (Sec. IV-B.3: per-layer latency is dominated by loading that layer's weights).  So every
// projection here is one persistent kernel that streams the weight matrix exactly once with
// 16-byte no-allocate loads, keeps the (tiny) activations in shared memory as bf16, accumulates
// in fp32 registers, reduces with warp shuffles, and runs the operation's epilogue in place:
//   QkvOp      RMSNorm prologue; rotary embedding of q and k; K/V appended to the cache
//   ResidOp    h += W x                      (attention output projection, MLP down projection)
//   GateUpOp   RMSNorm prologue; silu(W_g m) * (W_u m)
//   HeadOp     RMSNorm prologue; logits of one modality's id range and their arg max
// A "group" is R weight rows whose results one epilogue call needs together (a rotary pair, a
// gate/up pair).  A group is processed by a team of `ks` warps that split the inner dimension.
#pragma once

#include "sparsk_common.cuh"

namespace sparsk {

constexpr int GV_THREADS = 512;
constexpr int GV_WARPS = GV_THREADS / 32;
constexpr int GV_MC = 4;  // activation rows per pass

struct GvIn {
    const float *h;      // fp32 rows to normalise (NORM prologue)          [*, K]
    const bf16 *x;       // bf16 rows used as they are (plain prologue)      [*, K]
    const bf16 *gain;    // RMSNorm gain [K]
    const int *row_idx;  // optional indirection: activation row of pass-row i
    float eps;
    int K;       // inner dimension
    int n_rows;  // activation rows in this launch (all passes)
    int ks;      // warps per team (power of two <= 16)
};

// ------------------------------------------------------------------ prologues
template <int M, bool NORM>
__device__ __forceinline__ void gv_load_act(const GvIn &in, int m0, int mrows, bf16 *act, float *red)
{
    const int K = in.K, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    for (int m = 0; m < M; m++) {
        bf16 *dst = act + (size_t)m * K;
        if (m >= mrows) {
            for (int i = tid * 8; i < K; i += GV_THREADS * 8) *reinterpret_cast<uint4 *>(dst + i) = make_uint4(0, 0, 0, 0);
            continue;
        }
        const int row = in.row_idx ? in.row_idx[m0 + m] : (m0 + m);
        if (NORM) {
            const float *src = in.h + (size_t)row * K;
            float ss = 0.f;
            for (int i = tid * 4; i < K; i += GV_THREADS * 4) {
                float4 v = *reinterpret_cast<const float4 *>(src + i);
                ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
            }
            ss = warp_sum(ss);
            if (lane == 0) red[warp] = ss;
            __syncthreads();
            float tot = 0.f;
#pragma unroll
            for (int w = 0; w < GV_WARPS; w++) tot += red[w];
            __syncthreads();
            const float inv = rsqrtf(tot / (float)K + in.eps);
            for (int i = tid * 8; i < K; i += GV_THREADS * 8) {
                float4 a = *reinterpret_cast<const float4 *>(src + i);
                float4 b = *reinterpret_cast<const float4 *>(src + i + 4);
                float g[8];
                unpack8(*reinterpret_cast<const uint4 *>(in.gain + i), g);
                uint4 o;
                o.x = pack_bf16x2(a.x * inv * g[0], a.y * inv * g[1]);
                o.y = pack_bf16x2(a.z * inv * g[2], a.w * inv * g[3]);
                o.z = pack_bf16x2(b.x * inv * g[4], b.y * inv * g[5]);
                o.w = pack_bf16x2(b.z * inv * g[6], b.w * inv * g[7]);
                *reinterpret_cast<uint4 *>(dst + i) = o;
            }
        } else {
            const bf16 *src = in.x + (size_t)row * K;
            for (int i = tid * 8; i < K; i += GV_THREADS * 8)
                *reinterpret_cast<uint4 *>(dst + i) = *reinterpret_cast<const uint4 *>(src + i);
        }
    }
}

// ------------------------------------------------------------------ inner product
template <int R, int M>
__device__ __forceinline__ void gv_consume(const uint4 (&wv)[R], const bf16 *act, int K, int k, float (&acc)[R][M])
{
    float w[R][8];
#pragma unroll
    for (int r = 0; r < R; r++) unpack8(wv[r], w[r]);
#pragma unroll
    for (int m = 0; m < M; m++) {
        float a[8];
        unpack8(*reinterpret_cast<const uint4 *>(act + (size_t)m * K + k), a);
#pragma unroll
        for (int r = 0; r < R; r++) {
#pragma unroll
            for (int j = 0; j < 8; j++) acc[r][m] = fmaf(w[r][j], a[j], acc[r][m]);
        }
    }
}

// This warp's share of the inner dimension: 256-element chunks kw, kw+ks, kw+2ks, ...
// U chunks are loaded before any is consumed, so every lane keeps U*R 16-byte loads in flight.
template <int R, int M>
__device__ __forceinline__ void gv_accum(const bf16 *const (&wrow)[R], const bf16 *act, int K, int kw, int ks,
                                         int lane, float (&acc)[R][M])
{
    constexpr int U = 8 / R;
    const int nchunk = (K + 255) >> 8;
    for (int c = kw; c < nchunk; c += U * ks) {
        uint4 w[U][R];
        int k[U];
#pragma unroll
        for (int u = 0; u < U; u++) {
            k[u] = ((c + u * ks) << 8) + lane * 8;
            const bool p = (c + u * ks) < nchunk && k[u] < K;
            if (!p) k[u] = -1;
#pragma unroll
            for (int r = 0; r < R; r++) w[u][r] = p ? ld_stream16(wrow[r] + k[u]) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int u = 0; u < U; u++)
            if (k[u] >= 0) gv_consume<R, M>(w[u], act, K, k[u], acc);
    }
}

// ------------------------------------------------------------------ kernel
template <class Op, int R, int M, bool NORM>
__global__ void __launch_bounds__(GV_THREADS, 1) gemv_kernel(Op op, GvIn in)
{
    extern __shared__ __align__(16) unsigned char gv_smem[];
    bf16 *act = reinterpret_cast<bf16 *>(gv_smem);
    float *part = reinterpret_cast<float *>(gv_smem + (((size_t)M * in.K * 2 + 15) & ~(size_t)15));  // [2][warps][R*M]
    __shared__ float red[GV_WARPS];

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int ks = in.ks, tpc = GV_WARPS / ks, team = warp / ks, kw = warp % ks;
    const int n_groups = op.n_groups();
    const int m0 = blockIdx.y * GV_MC;
    const int mrows = min(M, in.n_rows - m0);

    // The weights do not depend on the previous kernel: pull this warp's first rows towards L2
    // while the previous kernel drains, then wait for its results.
    {
        const int g = team * gridDim.x + blockIdx.x;
        if (g < n_groups && blockIdx.y == 0) {
#pragma unroll
            for (int r = 0; r < R; r++) {
                const bf16 *p = op.row_ptr(g, r);
                for (int c = kw; c < ((in.K + 255) >> 8); c += ks) {
                    const int k = (c << 8) + lane * 8;
                    if ((lane & 7) == 0 && k < in.K) prefetch_l2(p + k);
                }
            }
        }
    }
    griddep_launch();
    griddep_wait();

    gv_load_act<M, NORM>(in, m0, mrows, act, red);
    __syncthreads();

    typename Op::State st;
    op.init(st);
    const int per_iter = gridDim.x * tpc;
    const int iters = (n_groups + per_iter - 1) / per_iter;
    for (int it = 0; it < iters; it++) {
        // consecutive groups go to different CTAs, so a partial last round spreads over all SMs
        const int g = it * per_iter + team * gridDim.x + blockIdx.x;
        const bool active = g < n_groups;
        float acc[R][M];
#pragma unroll
        for (int r = 0; r < R; r++)
#pragma unroll
            for (int m = 0; m < M; m++) acc[r][m] = 0.f;
        if (active) {
            const bf16 *wrow[R];
#pragma unroll
            for (int r = 0; r < R; r++) wrow[r] = op.row_ptr(g, r);
            gv_accum<R, M>(wrow, act, in.K, kw, ks, lane, acc);
        }
#pragma unroll
        for (int r = 0; r < R; r++)
#pragma unroll
            for (int m = 0; m < M; m++) acc[r][m] = warp_sum(acc[r][m]);

        float v[R];
        if (ks == 1) {
#pragma unroll
            for (int r = 0; r < R; r++) {
                v[r] = acc[r][0];
#pragma unroll
                for (int m = 1; m < M; m++)
                    if (lane == m) v[r] = acc[r][m];
            }
            if (active && lane < mrows) op.finish(g, m0 + lane, v, st);
        } else {
            float *pp = part + (size_t)(it & 1) * GV_WARPS * R * M;
            if (lane == 0) {
#pragma unroll
                for (int r = 0; r < R; r++)
#pragma unroll
                    for (int m = 0; m < M; m++) pp[warp * R * M + r * M + m] = acc[r][m];
            }
            __syncthreads();
            if (active && kw == 0 && lane < mrows) {
#pragma unroll
                for (int r = 0; r < R; r++) {
                    float s = 0.f;
                    for (int w = 0; w < ks; w++) s += pp[(warp + w) * R * M + r * M + lane];
                    v[r] = s;
                }
                op.finish(g, m0 + lane, v, st);
            }
        }
    }
    op.final(st, m0, mrows);
}

// ------------------------------------------------------------------ operations

// Fused RMSNorm + q/k/v projection + rotary embedding + cache append.
// Groups (R = 2P rows): P consecutive rotary pairs (i, i + hd/2) of one q or k head, or R
// consecutive rows of v.
template <int R>
struct QkvOp {
    struct State {};
    const bf16 *wq, *wk, *wv;
    float *q_out;             // [rows][Hq*hd] fp32
    kv_t *kc, *vc;            // this layer's cache: [slot][Hkv][S][hd]
    const float2 *rope;       // [S][hd/2] (cos, sin)
    const int *row_slot, *row_pos;
    int d, Hq, Hkv, hd, S;
    static constexpr int P = R / 2;

    __device__ int gq() const { return Hq * (hd / 2) / P; }
    __device__ int gk() const { return Hkv * (hd / 2) / P; }
    __device__ int n_groups() const { return gq() + gk() + Hkv * hd / R; }
    __device__ void init(State &) const {}
    __device__ const bf16 *row_ptr(int g, int r) const
    {
        const int half = hd / 2, per_head = half / P;
        if (g < gq() + gk()) {
            const bool isq = g < gq();
            const int gg = isq ? g : g - gq();
            const int head = gg / per_head, i0 = (gg % per_head) * P;
            const int row = head * hd + i0 + (r % P) + (r / P) * half;
            return (isq ? wq : wk) + (size_t)row * d;
        }
        const int gg = g - gq() - gk();
        return wv + (size_t)(gg * R + r) * d;
    }
    __device__ void finish(int g, int m, const float *v, State &) const
    {
        const int half = hd / 2, per_head = half / P;
        const int slot = row_slot[m], pos = row_pos[m];
        if (g < gq() + gk()) {
            const bool isq = g < gq();
            const int gg = isq ? g : g - gq();
            const int head = gg / per_head, i0 = (gg % per_head) * P;
#pragma unroll
            for (int p = 0; p < P; p++) {
                const float2 cs = rope[(size_t)pos * half + i0 + p];
                const float a = v[p], b = v[P + p];
                const float ra = a * cs.x - b * cs.y, rb = b * cs.x + a * cs.y;
                if (isq) {
                    float *dst = q_out + (size_t)m * Hq * hd + head * hd + i0 + p;
                    dst[0] = ra;
                    dst[half] = rb;
                } else {
                    kv_t *dst = kc + (((size_t)slot * Hkv + head) * S + pos) * hd + i0 + p;
                    dst[0] = to_kv(ra);
                    dst[half] = to_kv(rb);
                }
            }
        } else {
            const int row0 = (g - gq() - gk()) * R;
            const int head = row0 / hd, i0 = row0 % hd;
            kv_t *dst = vc + (((size_t)slot * Hkv + head) * S + pos) * hd + i0;
#pragma unroll
            for (int r = 0; r < R; r++) dst[r] = to_kv(v[r]);
        }
    }
    __device__ void final(State &, int, int) const {}
};

// h[m][row] += W[row] . x[m]
template <int R>
struct ResidOp {
    struct State {};
    const bf16 *w;
    float *h;  // [rows][n_out]
    int K, n_out;
    __device__ int n_groups() const { return (n_out + R - 1) / R; }
    __device__ void init(State &) const {}
    __device__ const bf16 *row_ptr(int g, int r) const { return w + (size_t)min(g * R + r, n_out - 1) * K; }
    __device__ void finish(int g, int m, const float *v, State &) const
    {
#pragma unroll
        for (int r = 0; r < R; r++)
            if (g * R + r < n_out) h[(size_t)m * n_out + g * R + r] += v[r];
    }
    __device__ void final(State &, int, int) const {}
};

// u[m][i] = silu(W_g[i] . x) * (W_u[i] . x); groups hold P gate rows and the matching up rows.
template <int R>
struct GateUpOp {
    struct State {};
    const bf16 *wg, *wu;
    bf16 *u;  // [rows][F]
    int d, F;
    static constexpr int P = R / 2;
    __device__ int n_groups() const { return (F + P - 1) / P; }
    __device__ void init(State &) const {}
    __device__ const bf16 *row_ptr(int g, int r) const
    {
        const int i = min(g * P + (r % P), F - 1);
        return ((r / P) ? wu : wg) + (size_t)i * d;
    }
    __device__ void finish(int g, int m, const float *v, State &) const
    {
#pragma unroll
        for (int p = 0; p < P; p++) {
            const int i = g * P + p;
            if (i < F) {
                const float gt = v[p];
                u[(size_t)m * F + i] = __float2bfloat16(gt / (1.f + __expf(-gt)) * v[P + p]);
            }
        }
    }
    __device__ void final(State &, int, int) const {}
};

// Exit head: logits of ids [lo, hi) and their arg max (lowest id on ties), per sequence.
template <int R>
struct HeadOp {
    struct State {
        float best;
        int id;
    };
    const bf16 *w;           // head projection [V][d]
    const int *seq_of_row;   // sequence index of pass-row i
    unsigned long long *argmax;
    float *logits;           // optional [n_seq][V]
    int d, lo, hi, V;
    __device__ int n_groups() const { return (hi - lo + R - 1) / R; }
    __device__ void init(State &s) const
    {
        s.best = -INFINITY;
        s.id = 0x7fffffff;
    }
    __device__ const bf16 *row_ptr(int g, int r) const { return w + (size_t)min(lo + g * R + r, hi - 1) * d; }
    __device__ void finish(int g, int m, const float *v, State &s) const
    {
#pragma unroll
        for (int r = 0; r < R; r++) {
            const int id = lo + g * R + r;
            if (id < hi) {
                if (v[r] > s.best || (v[r] == s.best && id < s.id)) {
                    s.best = v[r];
                    s.id = id;
                }
                if (logits) logits[(size_t)seq_of_row[m] * V + id] = v[r];
            }
        }
    }
    __device__ void final(State &s, int m0, int mrows) const
    {
        // every thread that ran an epilogue holds a candidate for pass-row m0 + lane
        const int lane = threadIdx.x & 31;
        if (lane < mrows && s.id != 0x7fffffff) atomicMax(&argmax[seq_of_row[m0 + lane]], argmax_key(s.best, s.id));
    }
};

}  // namespace sparsk

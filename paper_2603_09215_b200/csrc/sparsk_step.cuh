// Step bookkeeping kernels: exit schedule, active-row compaction, embedding gather,
// pending-store traffic and the state update that ends a step.
#pragma once

#include "sparsk_common.cuh"

namespace sparsk {

// Layers a step runs (Sec. IV-B.1): in-chunk index c runs L layers iff c mod K == r, else e.
// text_exit 0: text (modality 0) always runs L; 1: text follows the rule too; 2: only text follows
// it and speech always runs L (Sec. V-E, row G10).  Text steps that follow the rule use their own
// period and phase (Kt, rt), speech steps (K, r): the two modalities may need different policies
// (Sec. V-E).  The host's mirror of the pending counts uses the same function.
struct SchedParams {
    int L, e, K, r, Kt, rt, text_exit;
};
__host__ __device__ inline int scheduled_depth(int modality, int c, const SchedParams &p)
{
    if (modality == 0 && p.text_exit == 0) return p.L;
    if (modality != 0 && p.text_exit == 2) return p.L;
    if (modality == 0) return (c % p.Kt == p.rt) ? p.L : p.e;
    return (c % p.K == p.r) ? p.L : p.e;
}

// ---------------------------------------------------------------------------------------
// Exit schedule (Sec. IV-B.1).  One thread per sequence.  Also latches the input token (clamped
// into the vocabulary, with a status bit if it was outside) and clears the sequence's argmax cell.
// ---------------------------------------------------------------------------------------
static __global__ void schedule_kernel(StepDesc sd, int n, const int *__restrict__ staged /*[3][n]*/,
                                const int *__restrict__ tokens_in, int vocab, SchedParams sp)
{
    griddep_wait();
    int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b == 0) sd.counts[CNT_NSEQ] = n;
    if (b >= n) return;
    int slot = staged[b], mod = staged[n + b], c = staged[2 * n + b];
    int depth = scheduled_depth(mod, c, sp);
    int tok = tokens_in[b];
    if (tok < 0 || tok >= vocab) {
        atomicOr(&sd.counts[CNT_STATUS], ST_BAD_TOKEN);
        tok = min(max(tok, 0), vocab - 1);
    }
    sd.slot[b] = slot;
    sd.modality[b] = mod;
    sd.counter[b] = c;
    sd.token[b] = tok;
    sd.depth[b] = depth;
    sd.argmax[b] = 0ull;
}

// Exclusive prefix sum over one value per thread of a 1024-thread block; returns the prefix
// and leaves the block total in *total (shared).
__device__ __forceinline__ int block_exscan(int v, int *warp_tot /*[32] shared*/, int *total)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += t;
    }
    if (lane == 31) warp_tot[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = warp_tot[lane];
        int winc = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xffffffffu, winc, o);
            if (lane >= o) winc += t;
        }
        warp_tot[lane] = winc - w;
        if (lane == 31) *total = winc;
    }
    __syncthreads();
    int res = warp_tot[warp] + inc - v;
    __syncthreads();
    return res;
}

// ---------------------------------------------------------------------------------------
// Active-row compaction.  Sequences that leave at layer e drop out of layers e+1..L; every
// full-depth sequence contributes its pending positions plus its current one (Algorithm 1,
// full-depth branch).  Prefix sums give each sequence its offset in the upper row list; four
// more give the per-(exit, modality) lists the head kernels read.  One block, n <= 1024.
// ---------------------------------------------------------------------------------------
static __global__ void __launch_bounds__(1024) compact_kernel(StepDesc sd, int n, const int *__restrict__ kv_len,
                                                       const int *__restrict__ pend_cnt, int L, int e,
                                                       int list_stride)
{
    __shared__ int warp_tot[32];
    __shared__ int total;
    griddep_wait();
    const int b = threadIdx.x;
    const bool on = b < n;
    int slot = 0, depth = 0, mod = 0, len = 0, pend = 0;
    if (on) {
        slot = sd.slot[b];
        depth = sd.depth[b];
        mod = sd.modality[b];
        len = kv_len[slot];
        pend = pend_cnt[slot];
        sd.lo_pos[b] = len;
        sd.lo_grp_row0[b] = b;
        sd.lo_grp_nrows[b] = 1;
    }
    // a sequence needs the upper pass iff it runs L layers and L > e
    const bool full = on && depth == L;
    const bool upper = full && e < L;
    const int cnt = upper ? pend + 1 : 0;
    const int off = block_exscan(cnt, warp_tot, &total);
    if (b == 0) sd.counts[CNT_MUP] = total;
    const int grp = block_exscan(upper ? 1 : 0, warp_tot, &total);
    if (b == 0) sd.counts[CNT_NGRP] = total;
    if (on) sd.cur_row[b] = upper ? off + cnt - 1 : -1;
    if (upper) {
        sd.up_grp_row0[grp] = off;
        sd.up_grp_nrows[grp] = cnt;
        for (int j = 0; j < cnt; j++) {
            sd.up_slot[off + j] = slot;
            sd.up_pos[off + j] = len - pend + j;  // pending positions are the last `pend` ones
            sd.up_src[off + j] = (j < pend) ? j : -1 - b;
        }
    }
    // lists: 0 = early/text, 1 = early/speech, 2 = full/text, 3 = full/speech
#pragma unroll
    for (int l = 0; l < 4; l++) {
        const bool in = on && ((l >> 1) == (full ? 1 : 0)) && ((l & 1) == (mod ? 1 : 0));
        const int idx = block_exscan(in ? 1 : 0, warp_tot, &total);
        if (b == 0) sd.counts[CNT_LIST0 + l] = total;
        if (in) {
            sd.list_seq[l * list_stride + idx] = b;
            // hidden row the head reads: lower row b, or the sequence's current upper row
            sd.list_row[l * list_stride + idx] = (full && e < L) ? off + cnt - 1 : b;
        }
    }
}

// h^(0) = E[token]  (Sec. III), fp32 residual stream.
static __global__ void embed_kernel(const int *__restrict__ tokens, const bf16 *__restrict__ embed,
                             float *__restrict__ h, int n, int d, int vocab, int *__restrict__ status)
{
    griddep_wait();
    const int row = blockIdx.x;
    if (row >= n) return;
    int tok = tokens[row];
    if (tok < 0 || tok >= vocab) {  // never read outside the table; the host reports the flag
        if (threadIdx.x == 0) atomicOr(status, ST_BAD_TOKEN);
        tok = min(max(tok, 0), vocab - 1);
    }
    const bf16 *src = embed + (size_t)tok * d;
    for (int i = threadIdx.x * 8; i < d; i += blockDim.x * 8) {
        float f[8];
        unpack8(*reinterpret_cast<const uint4 *>(src + i), f);
        float4 *dst = reinterpret_cast<float4 *>(h + (size_t)row * d + i);
        dst[0] = make_float4(f[0], f[1], f[2], f[3]);
        dst[1] = make_float4(f[4], f[5], f[6], f[7]);
    }
}

// Early-exit rows: h^(e) goes to the pending store (Algorithm 1, early-exit branch).
static __global__ void stash_kernel(StepDesc sd, const float *__restrict__ h_lo, float *__restrict__ pend_h,
                             const int *__restrict__ pend_cnt, int n, int d, int L, int max_pending)
{
    griddep_wait();
    const int b = blockIdx.x;
    if (b >= n || sd.depth[b] == L) return;
    const int slot = sd.slot[b];
    const int j = pend_cnt[slot];
    if (j >= max_pending) return;  // the host refuses such a step before launching
    const float4 *src = reinterpret_cast<const float4 *>(h_lo + (size_t)b * d);
    float4 *dst = reinterpret_cast<float4 *>(pend_h + ((size_t)slot * max_pending + j) * d);
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) dst[i] = src[i];
}

// Upper rows: h^(e) of pending positions comes from the pending store, of the current
// position from the lower pass.
static __global__ void gather_upper_kernel(StepDesc sd, const float *__restrict__ h_lo,
                                    const float *__restrict__ pend_h, float *__restrict__ h_up, int d,
                                    int max_pending)
{
    griddep_wait();
    const int row = blockIdx.x;
    if (row >= sd.counts[CNT_MUP]) return;
    const int src = sd.up_src[row];
    const float *from = (src >= 0) ? pend_h + ((size_t)sd.up_slot[row] * max_pending + src) * d
                                   : h_lo + (size_t)(-1 - src) * d;
    const float4 *s4 = reinterpret_cast<const float4 *>(from);
    float4 *d4 = reinterpret_cast<float4 *>(h_up + (size_t)row * d);
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) d4[i] = s4[i];
}

// Last layer of the upper pass: pending rows only need their K/V there (nothing reads their
// h^(L): Algorithm 1's full-depth branch takes the token from the current position alone), so
// after the K/V projection the layer goes on with one row per full-depth sequence.  Group g's
// current row is the last row of the group: its residual stream and its query move to row g of
// the compact buffers, with its slot and position.
static __global__ void take_current_kernel(StepDesc sd, const float *__restrict__ h_up, const float *__restrict__ q_up,
                                    float *__restrict__ h_last, float *__restrict__ q_last,
                                    int *__restrict__ last_slot, int *__restrict__ last_pos, int d, int qd)
{
    griddep_wait();
    const int g = blockIdx.x;
    if (g >= sd.counts[CNT_NGRP]) return;
    const int row = sd.up_grp_row0[g] + sd.up_grp_nrows[g] - 1;
    if (threadIdx.x == 0) {
        last_slot[g] = sd.up_slot[row];
        last_pos[g] = sd.up_pos[row];
    }
    const float4 *hs = reinterpret_cast<const float4 *>(h_up + (size_t)row * d);
    float4 *hd4 = reinterpret_cast<float4 *>(h_last + (size_t)g * d);
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) hd4[i] = hs[i];
    const float4 *qs = reinterpret_cast<const float4 *>(q_up + (size_t)row * qd);
    float4 *qd4 = reinterpret_cast<float4 *>(q_last + (size_t)g * qd);
    for (int i = threadIdx.x; i < qd / 4; i += blockDim.x) qd4[i] = qs[i];
}
// ... and h^(L) of the current rows goes back to where the heads read it.
static __global__ void put_current_kernel(StepDesc sd, const float *__restrict__ h_last, float *__restrict__ h_up, int d)
{
    griddep_wait();
    const int g = blockIdx.x;
    if (g >= sd.counts[CNT_NGRP]) return;
    const int row = sd.up_grp_row0[g] + sd.up_grp_nrows[g] - 1;
    const float4 *s4 = reinterpret_cast<const float4 *>(h_last + (size_t)g * d);
    float4 *d4 = reinterpret_cast<float4 *>(h_up + (size_t)row * d);
    for (int i = threadIdx.x; i < d / 4; i += blockDim.x) d4[i] = s4[i];
}

// ---------------------------------------------------------------------------------------
// Confidence-based exit (Sec. V-B, compared method 3): after a layer's head has left the logits
// of the candidate rows in `logits` ([seq][V]), one block per row computes the entropy (natural
// logarithm) of softmax over the row's modality range [lo, hi): with m = max z, S = sum e^(z-m),
// T = sum (z-m) e^(z-m):  H = ln S - T / S.  Two passes over a row that sits in the L2.
// ---------------------------------------------------------------------------------------
static __global__ void __launch_bounds__(1024) entropy_kernel(const float *__restrict__ logits, const int *__restrict__ rows,
                                                       const int *__restrict__ row_mod, int n, int V, int Vt,
                                                       float *__restrict__ ent_out)
{
    __shared__ float red[32], red2[32];
    griddep_wait();
    const int i = blockIdx.x;
    if (i >= n) return;
    const int b = rows[i];
    const int lo = row_mod[i] ? Vt : 0, hi = row_mod[i] ? V : Vt;
    const float *z = logits + (size_t)b * V;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float mx = -INFINITY;
    for (int k = lo + threadIdx.x; k < hi; k += blockDim.x) mx = fmaxf(mx, z[k]);
    mx = warp_max(mx);
    if (lane == 0) red[warp] = mx;
    __syncthreads();
    mx = red[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); w++) mx = fmaxf(mx, red[w]);
    __syncthreads();
    float S = 0.f, T = 0.f;
    for (int k = lo + threadIdx.x; k < hi; k += blockDim.x) {
        const float x = z[k] - mx, e = __expf(x);
        S += e;
        T += x * e;
    }
    S = warp_sum(S);
    T = warp_sum(T);
    if (lane == 0) {
        red[warp] = S;
        red2[warp] = T;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float s = 0.f, t = 0.f;
        for (int w = 0; w < (int)(blockDim.x >> 5); w++) {
            s += red[w];
            t += red2[w];
        }
        ent_out[i] = hi > lo ? logf(s) - t / s : 0.f;
    }
}

// Rows between the residual-stream buffers of a pass and their homes.  Row i of `buf` belongs to
// sequence index seq[i] of the step; src[i] >= 0: pending position src[i] of that sequence's
// slot (pending store), src[i] < 0: the sequence's current position (row seq[i] of h_lo).
// to_buf = 1 gathers, 0 scatters back.
static __global__ void rows_move_kernel(float *__restrict__ buf, float *__restrict__ h_lo, float *__restrict__ pend_h,
                                 const int *__restrict__ row_slot, const int *__restrict__ row_seq,
                                 const int *__restrict__ row_src, int n, int d, int max_pending, int to_buf)
{
    griddep_wait();
    const int i = blockIdx.x;
    if (i >= n) return;
    const int src = row_src[i];
    float *home = src >= 0 ? pend_h + ((size_t)row_slot[i] * max_pending + src) * d : h_lo + (size_t)row_seq[i] * d;
    float4 *a = reinterpret_cast<float4 *>(buf + (size_t)i * d), *b = reinterpret_cast<float4 *>(home);
    for (int k = threadIdx.x; k < d / 4; k += blockDim.x) {
        if (to_buf) a[k] = b[k];
        else b[k] = a[k];
    }
}

// Clears the arg-max cells of the listed sequences (a head is about to be consulted again).
static __global__ void clear_keys_kernel(unsigned long long *__restrict__ keys, const int *__restrict__ rows, int n)
{
    griddep_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) keys[rows[i]] = 0ull;
}

// End of step: emit tokens and depths, advance lengths, grow or clear the pending sets.
static __global__ void finish_kernel(StepDesc sd, int n, int *__restrict__ kv_len, int *__restrict__ pend_cnt,
                              int *__restrict__ next_tokens, int *__restrict__ exit_depths, int L)
{
    griddep_wait();
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= n) return;
    const int slot = sd.slot[b], depth = sd.depth[b];
    next_tokens[b] = (int)(0xffffffffu - (uint32_t)(sd.argmax[b] & 0xffffffffull));
    exit_depths[b] = depth;
    kv_len[slot] += 1;
    pend_cnt[slot] = (depth == L) ? 0 : pend_cnt[slot] + 1;
}

// Parity hooks: copy the hidden state each head read; pre-fill the logits with -inf.
static __global__ void debug_hidden_kernel(StepDesc sd, const float *__restrict__ h_lo,
                                    const float *__restrict__ h_up, float *__restrict__ out, int n, int d)
{
    griddep_wait();
    const int b = blockIdx.x;
    if (b >= n) return;
    const int cr = sd.cur_row[b];
    const float *from = (cr >= 0) ? h_up + (size_t)cr * d : h_lo + (size_t)b * d;
    for (int i = threadIdx.x; i < d; i += blockDim.x) out[(size_t)b * d + i] = from[i];
}
static __global__ void fill_kernel(float *__restrict__ p, size_t n, float v)
{
    griddep_wait();
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
        p[i] = v;
}

// Prefill bookkeeping: rows of one chunk of one prompt.
static __global__ void prefill_rows_kernel(int *__restrict__ row_slot, int *__restrict__ row_pos,
                                    int *__restrict__ grp_row0, int *__restrict__ grp_nrows, int slot,
                                    int pos0, int n)
{
    griddep_wait();
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        grp_row0[0] = 0;
        grp_nrows[0] = n;
    }
    if (i < n) {
        row_slot[i] = slot;
        row_pos[i] = pos0 + i;
    }
}
static __global__ void set_int_kernel(int *p, int v)
{
    griddep_wait();
    *p = v;
}

// Cache import/export: [n][Hkv*hd] <-> [Hkv][S][hd] of one (layer, slot), fp16 on both sides.
static __global__ void kv_copy_kernel(kv_t *__restrict__ cache_k, kv_t *__restrict__ cache_v, kv_t *ext_k,
                               kv_t *ext_v, int first_pos, int n, int Hkv, int hd, int S, int to_cache)
{
    griddep_wait();
    const size_t total = (size_t)n * Hkv * hd;
    for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total;
         i += (size_t)gridDim.x * blockDim.x) {
        const int e = (int)(i % hd);
        const int hk = (int)((i / hd) % Hkv);
        const int t = (int)(i / ((size_t)hd * Hkv));
        const size_t c = ((size_t)hk * S + first_pos + t) * hd + e;
        if (to_cache) {
            cache_k[c] = ext_k[i];
            cache_v[c] = ext_v[i];
        } else {
            ext_k[i] = cache_k[c];
            ext_v[i] = cache_v[c];
        }
    }
}

}  // namespace sparsk

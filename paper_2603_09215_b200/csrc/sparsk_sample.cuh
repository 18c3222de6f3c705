// Nucleus (top-p) sampling with temperature over the id range of each sequence's modality
// (Sec. V-A: the 28-layer backbone decodes with temperature 0.7, top_p 0.9; the other backbone
// greedily, which is the arg max the heads already produce).
//
// No sort.  With w_i = exp((z_i - max z) / T):
//   1. the nucleus is every id whose w exceeds a threshold t, plus the first k ids (by id) whose
//      w equals t, where t is the largest value with  sum{w >= t} >= top_p * sum{w};
//   2. the drawn id is the one at which the cumulative mass, taken in decreasing w (equal w: lower
//      id first), first exceeds u * (kept mass); it has the largest w = v with sum{w >= v} > u * kept,
//      and among the ids with that w it is number floor((u * kept - sum{w > v}) / v).
// Both thresholds are found on the bit patterns of the positive floats (their unsigned order is
// their numeric order), four bits per pass: a pass sums the mass of the sixteen buckets that extend
// the prefix found so far.
//
// A row is read from memory once: every thread keeps its (up to 24) weights in registers for all
// twenty passes, ids in order (CTA, thread, register).  A pass adds each weight into the thread's
// own column of a [16][1024] shared-memory table (no conflicts, no atomics, a fixed order), the
// warps reduce the table, and, for ranges that need more than one CTA, the eight CTAs of a
// thread-block cluster combine their sixteen sums through distributed shared memory with one
// cluster barrier.  Ranges of up to 24,576 ids (the speech ranges) take one CTA per sequence,
// larger ones (the text ranges) a cluster of eight.  The uniform number u is the caller's (no
// generator on the device).
#pragma once

#include <cooperative_groups.h>

#include "sparsk_common.cuh"

namespace sparsk {

namespace cg = cooperative_groups;

constexpr int SP_THREADS = 1024;
constexpr int SP_CLUSTER = 8;
constexpr int SP_REGS = 24;                                      // weights a thread holds
constexpr int SP_CTA_RANGE = SP_THREADS * SP_REGS;               // ids one CTA holds: 24,576
constexpr int SP_MAX_RANGE = SP_CLUSTER * SP_CTA_RANGE;          // ids per modality: 196,608
constexpr int SP_SMEM = 16 * SP_THREADS * (int)sizeof(float);    // the per-thread bucket table

struct SampleArgs {
    const float *logits;         // [n][V]; only the modality's range of a row is read
    const float *uniforms;       // [n] in [0, 1)
    const int *modality;         // [n]: 0 text ids [0, Vt), else speech ids [Vt, Vt + Vs)
    unsigned long long *key_out; // optional [n]: the drawn id in the arg max key format
    int *token_out;              // optional [n]
    int V, Vt, Vs;
    int only_modality;           // rows of the other modality are left to another launch
    float inv_temperature, top_p;
};

struct SampleShared {
    float part[2][16];  // this CTA's sums of a pass, read by the whole cluster; double buffered
    float bcast[16];
    int i[32];
    int cnt_part, before_cta, all_eq;
};

// Combines the table's sixteen rows (one value per thread each) over the CTA and then over the
// cluster (sum, or max when use_max) in a fixed order; every thread gets all sixteen results.
// The caller has filled its column tab[c * SP_THREADS + tid]; `round` counts the calls.
template <int CL>
__device__ __forceinline__ void combine16(float *tab, float (&v)[16], bool use_max, SampleShared *sh, uint32_t &round)
{
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    __syncthreads();
    const int buf = round & 1;
    if (warp < 16) {  // warp c combines row c: 32 values per lane, then across the lanes
        const float *row = tab + warp * SP_THREADS;
        float x = row[lane];
#pragma unroll 8
        for (int i = 1; i < SP_THREADS / 32; i++) x = use_max ? fmaxf(x, row[i * 32 + lane]) : x + row[i * 32 + lane];
        x = use_max ? warp_max(x) : warp_sum(x);
        if (lane == 0) (CL > 1 ? sh->part[buf][warp] : sh->bcast[warp]) = x;
    }
    if (CL > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();  // also a barrier of this CTA
        if (warp < 16) {
            float x = use_max ? -INFINITY : 0.f;
            if (lane < CL) x = cluster.map_shared_rank(&sh->part[buf][0], lane)[warp];
            x = use_max ? warp_max(x) : warp_sum(x);
            if (lane == 0) sh->bcast[warp] = x;
        }
    }
    __syncthreads();
#pragma unroll
    for (int c = 0; c < 16; c++) v[c] = sh->bcast[c];
    // the table and bcast are next written after barriers that every thread must reach first
    round++;
}

// Largest bit pattern t with  mass{w >= t} >= target  (strict = false)  or  > target  (strict = true);
// `above` returns mass{w > t}, `at` returns mass{w == t}.
template <int CL>
__device__ __forceinline__ uint32_t threshold_search(float *tab, const float (&w)[SP_REGS], int n_mine, float target,
                                                     bool strict, float &above, float &at, SampleShared *sh,
                                                     uint32_t &round)
{
    uint32_t prefix = 0;
    float hi_mass = 0.f, bucket = 0.f;
    float *col = tab + threadIdx.x;
    for (int shift = 28; shift >= 0; shift -= 4) {
#pragma unroll
        for (int c = 0; c < 16; c++) col[c * SP_THREADS] = 0.f;  // (its last readers are behind a barrier)
        const uint32_t want = shift == 28 ? 0u : (prefix >> (shift + 4));
#pragma unroll
        for (int j = 0; j < SP_REGS; j++) {
            if (j < n_mine) {
                const uint32_t b = __float_as_uint(w[j]);
                if (shift == 28 || (b >> (shift + 4)) == want) col[((b >> shift) & 15u) * SP_THREADS] += w[j];
            }
        }
        float acc[16];
        combine16<CL>(tab, acc, false, sh, round);
        // the highest bucket whose mass, with everything above it, passes the target
        int pick = 0;
        float run = hi_mass;
        for (int c = 15; c >= 1; c--) {
            const float with = run + acc[c];
            if (strict ? with > target : with >= target) {
                pick = c;
                break;
            }
            run = with;
        }
        hi_mass = run;
        bucket = acc[pick];
        prefix |= (uint32_t)pick << shift;
    }
    above = hi_mass;
    at = bucket;
    return prefix;
}

// grid = n sequences x CL CTAs (cluster dimension CL when CL > 1); dynamic shared memory SP_SMEM.
template <int CL>
__global__ void __launch_bounds__(SP_THREADS, 1) nucleus_sample_kernel(SampleArgs a)
{
    extern __shared__ __align__(16) float sp_tab[];
    __shared__ SampleShared sh;
    griddep_wait();
    const int b = blockIdx.x / CL, rank = blockIdx.x % CL, tid = threadIdx.x;
    const int mod = a.modality[b] != 0;
    if (a.only_modality >= 0 && mod != a.only_modality) return;  // uniform over the cluster
    const int lo = mod ? a.Vt : 0, n = mod ? a.Vs : a.Vt;
    const float *z = a.logits + (size_t)b * a.V + lo;
    if (n < 1 || n > CL * SP_CTA_RANGE) {
        if (rank == 0 && tid == 0 && a.token_out) a.token_out[b] = -1;
        return;
    }
    // ids in order: (CTA, thread, register)
    const int per_thread = (n + CL * SP_THREADS - 1) / (CL * SP_THREADS);
    const int beg = min((rank * SP_THREADS + tid) * per_thread, n);
    const int n_mine = min(per_thread, n - beg);
    uint32_t round = 0;
    float *col = sp_tab + tid;

    float w[SP_REGS];
    float red[16];
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < SP_REGS; j++) {
        w[j] = j < n_mine ? z[beg + j] : -INFINITY;
        m = fmaxf(m, w[j]);
    }
#pragma unroll
    for (int c = 0; c < 16; c++) col[c * SP_THREADS] = c == 0 ? m : -INFINITY;
    combine16<CL>(sp_tab, red, true, &sh, round);
    m = red[0];
    float part = 0.f;
#pragma unroll
    for (int j = 0; j < SP_REGS; j++) {
        w[j] = j < n_mine ? expf((w[j] - m) * a.inv_temperature) : 0.f;
        part += w[j];
    }
#pragma unroll
    for (int c = 0; c < 16; c++) col[c * SP_THREADS] = c == 0 ? part : 0.f;
    combine16<CL>(sp_tab, red, false, &sh, round);
    const float total = red[0];

    // the nucleus: everything above t and the first k ids at t
    float above_t, at_t;
    const uint32_t t_bits = threshold_search<CL>(sp_tab, w, n_mine, a.top_p * total, false, above_t, at_t, &sh, round);
    const float t = __uint_as_float(t_bits);
    const int n_eq_t = (int)(t > 0.f ? at_t / t + 0.5f : 0.f);
    int k = n_eq_t;
    if (t > 0.f) {
        k = (int)ceilf((a.top_p * total - above_t) / t);
        k = max(1, min(k, max(n_eq_t, 1)));
    }
    const float kept = t > 0.f ? above_t + (float)k * t : above_t;

    // the draw
    const float u = fminf(fmaxf(a.uniforms[b], 0.f), 0.99999994f);
    const float ts = u * kept;
    float above_v, at_v;
    const uint32_t v_bits = threshold_search<CL>(sp_tab, w, n_mine, ts, true, above_v, at_v, &sh, round);
    const float v = __uint_as_float(v_bits);
    int q = v > 0.f ? (int)floorf((ts - above_v) / v) : 0;
    q = max(q, 0);
    if (v_bits == t_bits) q = min(q, k - 1);

    // the q-th id (in id order) whose weight is v
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < SP_REGS; j++) cnt += (j < n_mine && __float_as_uint(w[j]) == v_bits) ? 1 : 0;
    const int lane = tid & 31, warp = tid >> 5;
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) sh.i[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int s = sh.i[lane];
        int si = s;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, si, o);
            if (lane >= o) si += y;
        }
        sh.i[lane] = si - s;  // exclusive offset of each warp inside the CTA
        if (lane == 31) sh.cnt_part = si;
    }
    if (CL > 1) cg::this_cluster().sync();
    else __syncthreads();
    if (tid == 0) {
        int before_cta = 0, all = 0;
        for (int r = 0; r < CL; r++) {
            const int c = CL > 1 ? *cg::this_cluster().map_shared_rank(&sh.cnt_part, r) : sh.cnt_part;
            if (r < rank) before_cta += c;
            all += c;
        }
        sh.before_cta = before_cta;
        sh.all_eq = all;
    }
    __syncthreads();
    q = min(q, max(sh.all_eq - 1, 0));
    const int before = sh.before_cta + sh.i[warp] + incl - cnt;
    if (cnt > 0 && q >= before && q < before + cnt) {
        int seen = before, id = beg;
#pragma unroll
        for (int j = 0; j < SP_REGS; j++)
            if (j < n_mine && __float_as_uint(w[j]) == v_bits) {
                if (seen == q) id = beg + j;
                seen++;
            }
        const int token = lo + id;
        if (a.token_out) a.token_out[b] = token;
        if (a.key_out) a.key_out[b] = argmax_key(0.f, token);
    }
    if (CL > 1) cg::this_cluster().sync();  // no CTA leaves while another may still read its shared memory
}

// Launches for n rows: one CTA per row for the modalities whose range fits a CTA, a cluster of
// eight for the others; `has_text` / `has_speech` say which modalities occur among the rows.
inline cudaError_t launch_nucleus_sample(SampleArgs a, int n, bool has_text, bool has_speech, cudaStream_t st, bool pdl,
                                         int64_t *n_launches)
{
    static PerDevice<bool> ready_dev;
    bool &ready = ready_dev.here();
    if (!ready) {
        cudaError_t e = cudaFuncSetAttribute(nucleus_sample_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, SP_SMEM);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(nucleus_sample_kernel<SP_CLUSTER>, cudaFuncAttributeMaxDynamicSharedMemorySize, SP_SMEM);
        if (e != cudaSuccess) return e;
        ready = true;
    }
    for (int mod = 0; mod < 2; mod++) {
        if (!(mod ? has_speech : has_text)) continue;
        const int range = mod ? a.Vs : a.Vt;
        const int cl = range > SP_CTA_RANGE ? SP_CLUSTER : 1;
        a.only_modality = mod;
        cudaLaunchConfig_t cfg;
        memset(&cfg, 0, sizeof cfg);
        cfg.gridDim = dim3(n * cl);
        cfg.blockDim = dim3(SP_THREADS);
        cfg.dynamicSmemBytes = SP_SMEM;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        int na = 0;
        if (cl > 1) {
            attr[na].id = cudaLaunchAttributeClusterDimension;
            attr[na].val.clusterDim.x = cl;
            attr[na].val.clusterDim.y = 1;
            attr[na].val.clusterDim.z = 1;
            na++;
        }
        if (pdl) {
            attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[na].val.programmaticStreamSerializationAllowed = 1;
            na++;
        }
        cfg.attrs = attr;
        cfg.numAttrs = na;
        const cudaError_t e = cl > 1 ? cudaLaunchKernelEx(&cfg, nucleus_sample_kernel<SP_CLUSTER>, a)
                                     : cudaLaunchKernelEx(&cfg, nucleus_sample_kernel<1>, a);
        if (e != cudaSuccess) return e;
        if (n_launches) (*n_launches)++;
    }
    return cudaSuccess;
}

}  // namespace sparsk

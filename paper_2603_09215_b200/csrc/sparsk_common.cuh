// Shared device helpers of the SPAR-K decode kernels (sm_100a).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace sparsk {

typedef __nv_bfloat16 bf16;
// Element of the KV cache: IEEE half precision.  Weights and the activations that meet them are
// bfloat16, but a cached key or value is re-read by every later step, and at random
// initialisation its rounding error is amplified by every later layer: with 8 significant bits
// (bfloat16) the exit states of a 28-layer stack drift to 2 % from the fp64 reference once a few
// hundred positions of the cache are the decoder's own; the 11 bits of fp16 cost the same two
// bytes and leave 0.3 %.  Keys and values are O(1)..O(100) numbers, far inside the fp16 range;
// a value beyond it is stored as the largest finite fp16 number.
typedef __half kv_t;

// Row bookkeeping of one decode step, all device arrays inside the workspace.
// "Lower" rows are the step's sequences themselves (one row each, layers 1..e);
// "upper" rows are, for every sequence that runs full depth, its pending positions
// followed by its current position (layers e+1..L; Algorithm 1, full-depth branch).
struct StepDesc {
    int *slot, *modality, *counter, *token, *depth;  // [B]
    int *lo_pos;                                     // [B] position of the row = slot length
    int *lo_grp_row0, *lo_grp_nrows;                 // [B] identity groups (1 row each)
    int *up_slot, *up_pos, *up_src;                  // [R] src >= 0: pending index; < 0: lower row -1-src
    int *up_grp_row0, *up_grp_nrows;                 // [B] one group per full-depth sequence
    int *cur_row;                                    // [B] upper row of the current position, or -1
    int *list_seq, *list_row;                        // [4][B]: ee/text, ee/speech, full/text, full/speech
    int *counts;                                     // [8]: see CNT_* below
    unsigned long long *argmax;                      // [B] packed (logit, ~id)
};
enum { CNT_NSEQ = 0, CNT_MUP = 1, CNT_NGRP = 2, CNT_LIST0 = 3 /* ..6 */, CNT_STATUS = 7 };
enum { ST_BAD_TOKEN = 1, ST_TIMEOUT = 2 };

// Host side: a value kept once per device of the process.  Function attributes (dynamic
// shared-memory limits, occupancy answers) belong to a device, so "already set" is remembered
// for the device that is current, not for the process.
template <class T>
struct PerDevice {
    T v[64];
    T &here()
    {
        int dev = 0;
        cudaGetDevice(&dev);
        return v[(unsigned)dev & 63u];
    }
};

// Programmatic dependent launch.  A kernel lets the next one in the stream start as early as it
// can (launch_dependents, normally its first instruction) and touches nothing an earlier kernel
// writes before its own wait has returned (wait = the predecessor grid has completed and its
// writes are visible).  Every kernel here waits before it completes, so completion is transitive:
// when a kernel's wait returns, everything before it in the stream is done.  The early start is
// what lets a weight-streaming kernel issue its first weight copies (which depend on nothing)
// while a small kernel between two of them is still running.
__device__ __forceinline__ void griddep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void griddep_launch() { asm volatile("griddepcontrol.launch_dependents;"); }

// 16-byte streaming load that does not allocate in L1 (weights and cache lines are read once).
__device__ __forceinline__ uint4 ld_stream16(const void *p)
{
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}
__device__ __forceinline__ void prefetch_l2(const void *p)
{
    asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}

// bf16 pair packed in 32 bits -> two floats (element at the lower address first).
__device__ __forceinline__ float bf_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
__device__ __forceinline__ void unpack8(const uint4 &v, float (&f)[8])
{
    f[0] = bf_lo(v.x); f[1] = bf_hi(v.x); f[2] = bf_lo(v.y); f[3] = bf_hi(v.y);
    f[4] = bf_lo(v.z); f[5] = bf_hi(v.z); f[6] = bf_lo(v.w); f[7] = bf_hi(v.w);
}
__device__ __forceinline__ uint32_t pack_bf16x2(float a, float b)
{
    __nv_bfloat162 t = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&t);
}

// x = hi + lo with hi = bf16(x), lo = bf16(x - hi): two bf16 terms that carry 16 significant
// bits through a bf16 tensor-core product.
__device__ __forceinline__ void split_pair(float a, float b, uint32_t &hi, uint32_t &lo)
{
    hi = pack_bf16x2(a, b);  // one packed conversion, widened back with shifts
    lo = pack_bf16x2(a - bf_lo(hi), b - bf_hi(hi));
}
__device__ __forceinline__ void split8(const float (&v)[8], uint4 &hi, uint4 &lo)
{
    split_pair(v[0], v[1], hi.x, lo.x);
    split_pair(v[2], v[3], hi.y, lo.y);
    split_pair(v[4], v[5], hi.z, lo.z);
    split_pair(v[6], v[7], hi.w, lo.w);
}

__device__ __forceinline__ kv_t to_kv(float x) { return __float2half_rn(fminf(fmaxf(x, -65504.f), 65504.f)); }
// The same two-term form in fp16 (what multiplies the cache in the attention kernels): hi has 11
// significant bits, hi + lo about 22.
__device__ __forceinline__ uint32_t pack_h2(float a, float b)
{
    __half2 t = __floats2half2_rn(a, b);
    return *reinterpret_cast<uint32_t *>(&t);
}
__device__ __forceinline__ void split_pair_h(float a, float b, uint32_t &hi, uint32_t &lo)
{
    const __half2 h = __floats2half2_rn(a, b);
    const float2 f = __half22float2(h);
    hi = *reinterpret_cast<const uint32_t *>(&h);
    lo = pack_h2(a - f.x, b - f.y);
}
__device__ __forceinline__ void split8_h(const float (&v)[8], uint4 &hi, uint4 &lo)
{
    split_pair_h(v[0], v[1], hi.x, lo.x);
    split_pair_h(v[2], v[3], hi.y, lo.y);
    split_pair_h(v[4], v[5], hi.z, lo.z);
    split_pair_h(v[6], v[7], hi.w, lo.w);
}

__device__ __forceinline__ float warp_sum(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v)
{
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

// Order-preserving map float -> uint32, and the 64-bit key whose maximum is the largest logit
// with the lowest id among equals.
__device__ __forceinline__ uint32_t float_key(float f)
{
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ unsigned long long argmax_key(float logit, int id)
{
    return ((unsigned long long)float_key(logit) << 32) | (unsigned long long)(0xffffffffu - (uint32_t)id);
}

// Longest any in-kernel wait may last (wall clock); after it the waiter raises ST_TIMEOUT and leaves.
constexpr unsigned long long WAIT_TIMEOUT_NS = 2000000000ull;

// ------------------------------------------------------------------ mbarrier, TMA and timer wrappers
__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long global_ns()
{
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar)
{
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity)
{
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait for a phase of an mbarrier.  Returns false if the CTA is giving up (another
// thread did, or this wait outlasted `limit_ns`); the caller then leaves its loop.
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity, volatile int *giving_up, int *status,
                                          unsigned long long limit_ns = WAIT_TIMEOUT_NS)
{
    unsigned long long t0 = 0;
    for (uint32_t spin = 0;; ++spin) {
        if (mbar_test(bar, parity)) return true;
        if (spin > 64) __nanosleep(32);
        if ((spin & 255u) == 255u) {
            if (*giving_up) return false;
            const unsigned long long now = global_ns();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit_ns) {
                *giving_up = 1;
                if (status) atomicOr(status, ST_TIMEOUT);
                return false;
            }
        }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int x, int y)
{
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y)
        : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap *map, uint64_t *bar, int x, int y, int z)
{
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y), "r"(z)
        : "memory");
}

}  // namespace sparsk

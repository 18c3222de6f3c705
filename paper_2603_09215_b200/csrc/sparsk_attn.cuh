// Split-KV grouped-query attention over the ragged KV cache (flash-decoding) on tensor cores.
//
// A work item is (sequence group, block of 16 query vectors, kv head, KV split) and belongs to ONE
// warp.  A group is the block of rows of ONE sequence that a pass processes together: a single
// row in the lower pass, the pending positions plus the current one in the upper pass
// (Algorithm 1, full-depth branch: one causal block of at most K rows), a chunk of the prompt in
// prefill.  The query heads that share the kv head, for the rows of the group, form the M
// dimension of mma.sync m16n8k16 tiles, so one read of that head's K/V serves sixteen of them;
// row r of the group may look at positions <= pos0 + r (the causal mask of the block on top of
// the whole earlier cache).
//
// The warp keeps its sixteen query vectors as fp16 MMA fragments in registers (scaled by
// log2(e) / sqrt(hd), so that the softmax works in powers of two), streams 16-position K/V tiles
// of its split into a private shared-memory ring (no barrier wider than the warp anywhere),
// computes S = Q K^T and O += P V with fp16 MMAs and fp32 accumulators, and keeps an online
// softmax whose row maxima and sums are reduced with shuffles inside the four-lane groups that
// share an accumulator row.  Queries and softmax weights are rounded to fp16 once, like the cache
// they meet: the same 2^-12 relative error as a cached key or value carries.  The warp writes one
// unnormalised partial (acc, running max in log2 units turned back to natural-log units, running
// sum) per (row, query head, split); a second kernel merges the splits.
//
// Two forms of the ring: coalesced 16-byte cp.async copies into padded rows (callers that pass
// plain cache pointers: the stand-alone entry points, the persistent kernel), or one TMA box per
// tile and matrix with the 128-byte swizzle and an mbarrier per stage (the decode path, which
// holds tensor maps of its cache).  Two forms of an item: the one above, and a transposed one for
// groups of at most eight query vectors (a single row at up to eight query heads per kv head),
// where the positions are the M dimension and the work per tile halves (attn_item_t).
// Items are dealt to the warps of a persistent grid, each warp's first by its number and the rest,
// when there are more items than warps, from a ticket counter as warps finish: a warp's fixed cost
// per item is a few hundred instructions, which is what lets twelve warps per SM with one tile
// in flight each keep HBM busy where CTA-wide tiles with a cross-warp merge did not.
#pragma once

#include "sparsk_common.cuh"

namespace sparsk {

constexpr int AT_TP = 16;        // positions per tile
constexpr int AT_MAX_SPLITS = 32;
constexpr int AT_MIN_SPLIT = 64;
constexpr int AW_WARPS = 4;      // warps per CTA of the stand-alone kernel
constexpr int AW_NST = 2;        // ring stages per warp there (default; 3 is the other instantiation)

// How a launch cuts the work: blocks of 16 query vectors per group, and the KV range into
// splits so that every warp of the persistent grid gets a few items, none shorter than
// AT_MIN_SPLIT positions (unless forced), at most AT_MAX_SPLITS.
struct AttnPlan {
    int n_qblk, split_len, n_splits;
};
// `sum_len` is the total of the groups' prefix lengths when the caller knows it (0: assume every
// group is as long as the longest): with ragged lengths the splits past a short group's end are
// empty items, and sizing by the real total keeps the number of items with work near 1.75 per
// warp whatever the spread of the lengths (shorter items add set-up, longer ones a ragged end).
inline AttnPlan attn_plan(int n_workers, int n_groups, int max_grp_rows, int G, int Hkv, int max_len, int forced_split,
                          long sum_len = 0)
{
    AttnPlan p;
    const int nq = max_grp_rows * G;
    p.n_qblk = (nq + 15) / 16;
    int split = forced_split;
    if (split <= 0) {
        const long groups = n_groups < 1 ? 1 : n_groups;
        const long total = (sum_len > 0 ? sum_len : groups * (long)max_len) * p.n_qblk * Hkv;  // positions x heads to visit
        split = (int)(total * 4 / (7L * n_workers));  // 1.75 items per warp (measured best at 64 ragged sequences)
        if (split < AT_MIN_SPLIT) split = AT_MIN_SPLIT;
        if (split > max_len) split = max_len < 1 ? 1 : max_len;
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
// shared memory of one warp's K/V ring
inline size_t attn_warp_bytes(int head_dim, int stages) { return (size_t)stages * 2 * AT_TP * (head_dim + 8) * 2; }

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
    int max_groups;           // host bound on the number of groups (sizes the item space)
    // Dynamic dealing of items (optional): a counter that only ever grows.  With W warps and
    // n > W items, warp w starts on item w and ticket ticket_base + t stands for item W + t
    // (unsigned arithmetic, so the counter may wrap); every warp draws exactly one ticket beyond
    // its last item, so the launch adds n to the counter, which is how the host knows the next
    // launch's base without reading it.  With n <= W no ticket is drawn.  NULL: items are dealt
    // round-robin.
    unsigned *ticket;
    unsigned ticket_base;
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

// The TMA-fed form of a warp's ring: tiles arrive as tensor-map boxes of 16 positions with the
// 128-byte swizzle (no padding, one copy per tile and matrix instead of sixteen cp.async per
// lane), each stage with an mbarrier of its own whose phases run on across the warp's items.
struct AttnTma {
    const CUtensorMap *mk, *mv;  // this layer's K and V cache as rows of head_dim fp16 numbers
    uint64_t *bars;              // the warp's NS barriers
    uint32_t seq;                // tiles this warp has consumed so far (stage = seq mod NS)
    volatile int *giving_up;     // CTA-wide: a wait ran out
    int *status;                 // device status word
};
// Element offset of 16-byte chunk c of row `row` inside a swizzled tile: blocks of 16 rows x 64
// elements (one per 64 elements of the head dimension), chunk index XOR row mod 8.
template <int HD>
__device__ __forceinline__ int at_swz(int row, int c)
{
    return (HD > 64 ? (c >> 3) * (AT_TP * 64) : 0) + row * 64 + (((c & 7) ^ (row & 7)) << 3);
}

// What a warp knows of an item before it starts: who it is for, and the span of positions it reads.
struct AtItem {
    int qb, hk, sp, row0, nrows, slot, pos0;
    int nq;                          // query vectors of the group per kv head
    int w_beg, w_end, n_tiles, y0;   // positions [w_beg, w_end) in tiles of 16; first cache row of (slot, hk)
    bool valid;                      // false: not an item of this launch (no partial either)
};
// Item number idx of a launch -> descriptor.  Straight-line code: every load is clamped instead of
// skipped, so the loads of one level go out together.
__device__ __forceinline__ AtItem at_resolve(const AttnArgs &a, unsigned idx, unsigned n_items, int n_groups,
                                             const int *grp_row0, const int *grp_nrows, const int *row_slot,
                                             const int *row_pos)
{
    AtItem it;
    const int G = a.Hq / a.Hkv;
    unsigned t = idx < n_items ? idx : 0u;
    it.qb = (int)(t % a.n_qblk); t /= a.n_qblk;
    it.hk = (int)(t % a.Hkv); t /= a.Hkv;
    const int g = (int)(t % a.max_groups);
    it.sp = (int)(t / a.max_groups);
    bool ok = idx < n_items && g < n_groups;
    const int gc = ok ? g : 0;
    it.row0 = grp_row0[gc];
    it.nrows = grp_nrows[gc];
    ok = ok && it.row0 >= 0 && it.nrows >= 1 && it.row0 + it.nrows <= a.n_rows;
    const int rc = ok ? it.row0 : 0;
    it.slot = row_slot[rc];
    it.pos0 = row_pos[rc];
    it.nq = it.nrows * G;
    ok = ok && it.qb * 16 < it.nq && it.nq >= a.nq_min && it.nq <= a.nq_max;
    // positions the item may look at: its split, cut at the last query row's own position (and
    // at the cache itself: a row that points outside it reads nothing)
    const bool sane = it.slot >= 0 && it.slot < a.n_slots && it.pos0 >= 0;
    const int nq_here = min(16, it.nq - it.qb * 16);
    const int last_row = (it.qb * 16 + nq_here - 1) / G;
    const int kv_end_all = ok && sane ? min(it.pos0 + last_row + 1, a.S) : 0;
    it.w_beg = it.sp * a.split_len;
    it.w_end = min(it.w_beg + a.split_len, kv_end_all);
    it.n_tiles = it.w_end > it.w_beg ? (it.w_end - it.w_beg + AT_TP - 1) / AT_TP : 0;
    it.y0 = ((sane ? it.slot : 0) * a.Hkv + it.hk) * a.S;
    it.valid = ok;
    return it;
}
// A warp's K/V ring, in either form: `issue` starts the copies of tile t of the split
// [w_beg, w_end), `wait` blocks until tile t has landed (false: a bounded wait ran out) and says
// where it is, `release` hands the stage back and refills it, `finish` closes the item.
template <int HD, int NS, bool TMA>
struct AtRing {
    static constexpr int KP = HD + 8;          // padded row of the cp.async form
    static constexpr int TP = TMA ? HD : KP;   // row pitch of a tile in the ring
    static constexpr int CH = HD / 8;          // 16-byte chunks per row
    kv_t *wr;
    AttnTma *tm;
    const kv_t *kbase, *vbase;
    int w_beg, w_end, y0, lane, n_tiles;
    uint32_t seq0;

    __device__ __forceinline__ AtRing(const AttnArgs &a, const AtItem &it, kv_t *wr_, int lane_, AttnTma *tm_)
        : wr(wr_), tm(tm_), kbase(a.kc + (size_t)it.y0 * HD), vbase(a.vc + (size_t)it.y0 * HD), w_beg(it.w_beg),
          w_end(it.w_end), y0(it.y0), lane(lane_), n_tiles(it.n_tiles), seq0(TMA ? tm_->seq : 0u)
    {
    }

    // element offset of 16-byte chunk c of row `row` inside a tile
    __device__ __forceinline__ static int off(int row, int c) { return TMA ? at_swz<HD>(row, c) : row * KP + c * 8; }
    __device__ __forceinline__ int stage(int t) const { return (int)((seq0 + (uint32_t)t) % NS); }
    // TMA form: the tile whose first cache row is y, as tile number `seq` of this warp.  Rows past a
    // split's end arrive as whatever the cache holds there (zeros beyond the cache): the scores
    // mask them, the value rows are cleared after landing.
    __device__ __forceinline__ void issue_tma(int y, uint32_t seq) const
    {
        if (lane == 0) {
            const int st = (int)(seq % NS);
            kv_t *kt = wr + (size_t)st * 2 * AT_TP * TP, *vt = kt + AT_TP * TP;
            mbar_expect_tx(&tm->bars[st], 2u * AT_TP * HD * (uint32_t)sizeof(kv_t));
            if (HD > 64) {
                tma_load_3d(smem_u32(kt), tm->mk, &tm->bars[st], 0, y, 0);
                tma_load_3d(smem_u32(vt), tm->mv, &tm->bars[st], 0, y, 0);
            } else {
                tma_load_2d(smem_u32(kt), tm->mk, &tm->bars[st], 0, y);
                tma_load_2d(smem_u32(vt), tm->mv, &tm->bars[st], 0, y);
            }
        }
    }
    __device__ __forceinline__ void issue(int t) const
    {
        const int st = stage(t);
        kv_t *kt = wr + (size_t)st * 2 * AT_TP * TP, *vt = kt + AT_TP * TP;
        const int p0 = w_beg + t * AT_TP;
        if constexpr (TMA) {
            issue_tma(y0 + p0, seq0 + (uint32_t)t);
        } else {
#pragma unroll
            for (int i = lane; i < AT_TP * CH; i += 32) {
                const int r = i / CH, c = i % CH;
                const bool ok = p0 + r < w_end;                  // rows past the end are zero-filled
                const size_t o = (size_t)(ok ? p0 + r : w_beg) * HD + c * 8;
                cp_async16(&kt[r * KP + c * 8], kbase + o, ok ? 16 : 0);
                cp_async16(&vt[r * KP + c * 8], vbase + o, ok ? 16 : 0);
            }
        }
    }
    __device__ __forceinline__ void start() const
    {
        __syncwarp();  // the previous item's last reads of the ring are over
#pragma unroll
        for (int t = 0; t < NS; t++) {
            if (t < n_tiles) issue(t);
            if (!TMA) cp_async_commit();
        }
    }
    __device__ __forceinline__ bool wait(int t, const kv_t *&Kt, const kv_t *&Vt) const
    {
        const int st = stage(t);
        kv_t *kt = wr + (size_t)st * 2 * AT_TP * TP, *vt = kt + AT_TP * TP;
        if constexpr (TMA) {
            if (!mbar_wait(&tm->bars[st], ((seq0 + (uint32_t)t) / NS) & 1u, tm->giving_up, tm->status)) return false;
            const int p0 = w_beg + t * AT_TP;
            if (p0 + AT_TP > w_end) {
                // value rows past the end meet a weight of exactly zero, which must not meet a
                // NaN or an infinity: clear them
                const int nv = w_end - p0;
                for (int i = lane; i < (AT_TP - nv) * CH; i += 32)
                    *reinterpret_cast<uint4 *>(&vt[at_swz<HD>(nv + i / CH, i % CH)]) = make_uint4(0u, 0u, 0u, 0u);
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            }
        } else {
            cp_async_wait<NS - 1>();
        }
        __syncwarp();
        Kt = kt;
        Vt = vt;
        return true;
    }
    __device__ __forceinline__ void release(int t) const
    {
        __syncwarp();  // every lane is done with this stage: refill it
        if (t + NS < n_tiles) issue(t + NS);
        if (!TMA) cp_async_commit();
    }
    __device__ __forceinline__ void finish() const
    {
        if constexpr (TMA) tm->seq = seq0 + (uint32_t)n_tiles;
        else cp_async_wait<0>();
    }
};

__device__ __forceinline__ uint32_t movmatrix_t(uint32_t x)
{
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

// One item, by one warp: query vectors [16 qb, 16 qb + 16) of a group (rows row0 .. row0 + nrows - 1
// of slot `slot`, the first at position pos0), kv head hk, split sp.  `wr` is the warp's ring of
// NS stages.  Writes the item's partial.
// QREG: the query fragments stay in registers for the whole item (32 registers at head dimension
// 128); otherwise they are parked in `qs` ([16][HD + 8] of shared memory) and re-read per tile,
// for callers whose register budget is spoken for.
template <int HD, int NS, bool QREG, bool TMA = false>
__device__ __forceinline__ void attn_item(const AttnArgs &a, const AtItem &it, kv_t *wr, kv_t *qs, int lane,
                                          AttnTma *tm = nullptr)
{
    typedef AtRing<HD, NS, TMA> Ring;
    constexpr int KP = HD + 8;      // padded row of the parked queries: ldmatrix rows fall into distinct banks
    constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
    const int G = a.Hq / a.Hkv, splits = a.n_splits;
    const int qb = it.qb, hk = it.hk, sp = it.sp, row0 = it.row0, pos0 = it.pos0;
    const int nq = it.nq, q0 = qb * 16;
    const int nq_here = min(16, nq - q0);
    const int w_beg = it.w_beg, w_end = it.w_end, n_tiles = it.n_tiles;
    if (n_tiles == 0) {
        // an empty split: max = -inf, sum = 0 is all the merge looks at
        for (int qi = lane; qi < nq_here; qi += 32) {
            const int qg = q0 + qi;
            a.part_ml[((size_t)(row0 + qg / G) * a.Hq + hk * G + qg % G) * splits + sp] = make_float2(-INFINITY, 0.f);
        }
        return;
    }
    Ring ring(a, it, wr, lane, tm);
    ring.start();

    // the queries, as A fragments (row = lane / 4 and + 8, columns 2 (lane % 4) + {0, 1, 8, 9} of
    // every 16-column step), while the first tiles are on their way
    uint32_t qa[QREG ? HD / 16 : 1][4];
    const float qscale = rsqrtf((float)HD) * LOG2E;
    {
        const int qi0 = lane >> 2, qi1 = qi0 + 8, c0 = (lane & 3) * 2;
        const bool h0 = qi0 < nq_here && n_tiles > 0, h1 = qi1 < nq_here && n_tiles > 0;
        const int g0 = q0 + (h0 ? qi0 : 0), g1 = q0 + (h1 ? qi1 : 0);
        const size_t o0 = (size_t)(row0 + g0 / G) * a.Hq * HD + (hk * G + g0 % G) * HD + c0;
        const size_t o1 = (size_t)(row0 + g1 / G) * a.Hq * HD + (hk * G + g1 % G) * HD + c0;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ks++) {
            float2 x00 = make_float2(0.f, 0.f), x01 = x00, x10 = x00, x11 = x00;
            if (a.q32) {
                if (h0) {
                    x00 = *reinterpret_cast<const float2 *>(a.q32 + o0 + ks * 16);
                    x01 = *reinterpret_cast<const float2 *>(a.q32 + o0 + ks * 16 + 8);
                }
                if (h1) {
                    x10 = *reinterpret_cast<const float2 *>(a.q32 + o1 + ks * 16);
                    x11 = *reinterpret_cast<const float2 *>(a.q32 + o1 + ks * 16 + 8);
                }
            } else {
                if (h0) {
                    const uint32_t u0 = *reinterpret_cast<const uint32_t *>(a.q + o0 + ks * 16);
                    const uint32_t u1 = *reinterpret_cast<const uint32_t *>(a.q + o0 + ks * 16 + 8);
                    x00 = make_float2(bf_lo(u0), bf_hi(u0));
                    x01 = make_float2(bf_lo(u1), bf_hi(u1));
                }
                if (h1) {
                    const uint32_t u0 = *reinterpret_cast<const uint32_t *>(a.q + o1 + ks * 16);
                    const uint32_t u1 = *reinterpret_cast<const uint32_t *>(a.q + o1 + ks * 16 + 8);
                    x10 = make_float2(bf_lo(u0), bf_hi(u0));
                    x11 = make_float2(bf_lo(u1), bf_hi(u1));
                }
            }
            const uint32_t f0 = pack_h2(x00.x * qscale, x00.y * qscale), f1 = pack_h2(x10.x * qscale, x10.y * qscale);
            const uint32_t f2 = pack_h2(x01.x * qscale, x01.y * qscale), f3 = pack_h2(x11.x * qscale, x11.y * qscale);
            if (QREG) {
                qa[ks][0] = f0; qa[ks][1] = f1; qa[ks][2] = f2; qa[ks][3] = f3;
            } else {
                *reinterpret_cast<uint32_t *>(&qs[qi0 * KP + ks * 16 + c0]) = f0;
                *reinterpret_cast<uint32_t *>(&qs[qi1 * KP + ks * 16 + c0]) = f1;
                *reinterpret_cast<uint32_t *>(&qs[qi0 * KP + ks * 16 + c0 + 8]) = f2;
                *reinterpret_cast<uint32_t *>(&qs[qi1 * KP + ks * 16 + c0 + 8]) = f3;
            }
        }
        if (!QREG) __syncwarp();
    }

    float o[HD / 8][4], m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
    for (int nt = 0; nt < HD / 8; nt++)
#pragma unroll
        for (int e = 0; e < 4; e++) o[nt][e] = 0.f;
    // last position each of this thread's two accumulator rows may see
    int limit[2];
#pragma unroll
    for (int hf = 0; hf < 2; hf++) {
        const int qi = (lane >> 2) + hf * 8;
        limit[hf] = qi < nq_here ? pos0 + (q0 + qi) / G : -1;
    }
    const int lim_min = pos0 + q0 / G;  // the smallest limit among the item's query vectors

    for (int t = 0; t < n_tiles; t++) {
        const kv_t *Kt, *Vt;
        if (!ring.wait(t, Kt, Vt)) return;
        const int p0 = w_beg + t * AT_TP;

        // S = Q K^T for 16 positions, in log2 units; two accumulator chains
        float s[2][4], s2[2][4];
#pragma unroll
        for (int nt = 0; nt < 2; nt++)
#pragma unroll
            for (int e = 0; e < 4; e++) s[nt][e] = s2[nt][e] = 0.f;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ks += 2) {
            uint32_t kb[4], kb2[4];
            const int krow = (lane & 7) + ((lane >> 4) << 3), kch = (lane >> 3) & 1;
            ldsm_x4(kb, &Kt[Ring::off(krow, ks * 2 + kch)]);
            ldsm_x4(kb2, &Kt[Ring::off(krow, (ks + 1) * 2 + kch)]);
            if (QREG) {
                mma_f16(s[0], qa[ks], kb[0], kb[1]);
                mma_f16(s[1], qa[ks], kb[2], kb[3]);
                mma_f16(s2[0], qa[ks + 1], kb2[0], kb2[1]);
                mma_f16(s2[1], qa[ks + 1], kb2[2], kb2[3]);
            } else {
                uint32_t q1[4], q2[4];
                const int qoff = ((lane & 7) + ((lane >> 3) & 1) * 8) * KP + (lane >> 4) * 8;
                ldsm_x4(q1, &qs[qoff + ks * 16]);
                ldsm_x4(q2, &qs[qoff + (ks + 1) * 16]);
                mma_f16(s[0], q1, kb[0], kb[1]);
                mma_f16(s[1], q1, kb[2], kb[3]);
                mma_f16(s2[0], q2, kb2[0], kb2[1]);
                mma_f16(s2[1], q2, kb2[2], kb2[3]);
            }
        }
        // online softmax; P as the A operand of the second product.  A tile wholly inside what
        // every query vector of the item may see (all but the last of an item) needs no masking;
        // accumulator rows without a query vector then carry numbers nobody reads.
        const bool full = p0 + AT_TP <= w_end && p0 + AT_TP - 1 <= lim_min;
        uint32_t pa[4];
        float alpha[2];
#pragma unroll
        for (int hf = 0; hf < 2; hf++) {
            float v[4];
            float tmax = -INFINITY;
#pragma unroll
            for (int nt = 0; nt < 2; nt++)
#pragma unroll
                for (int e = 0; e < 2; e++) {
                    const int p = p0 + nt * 8 + (lane & 3) * 2 + e;
                    const bool ok = full || (p < w_end && p <= limit[hf]);
                    v[nt * 2 + e] = ok ? s[nt][hf * 2 + e] + s2[nt][hf * 2 + e] : -INFINITY;
                    tmax = fmaxf(tmax, v[nt * 2 + e]);
                }
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
            const float m_new = fmaxf(m_run[hf], tmax);
            float psum = 0.f;
            alpha[hf] = 1.f;
            if (m_new != -INFINITY) {
                alpha[hf] = exp2f(m_run[hf] - m_new);  // 2^(-inf) = 0 on the first live tile
#pragma unroll
                for (int i = 0; i < 4; i++) {
                    v[i] = exp2f(v[i] - m_new);
                    psum += v[i];
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; i++) v[i] = 0.f;
            }
            l_run[hf] = l_run[hf] * alpha[hf] + psum;  // per-thread share; lanes are summed at the end
            m_run[hf] = m_new;
            pa[hf] = pack_h2(v[0], v[1]);      // positions 0..7 of the tile
            pa[2 + hf] = pack_h2(v[2], v[3]);  // positions 8..15
        }
        // the accumulator is rescaled only when some row's maximum moved (after the first tiles
        // of an item that is rare)
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
            for (int nt = 0; nt < HD / 8; nt++) {
                o[nt][0] *= alpha[0];
                o[nt][1] *= alpha[0];
                o[nt][2] *= alpha[1];
                o[nt][3] *= alpha[1];
            }
        }
        // O += P V
#pragma unroll
        for (int np = 0; np < HD / 16; np++) {
            uint32_t vb[4];
            const int vrow = (lane & 7) + ((lane >> 3) & 1) * 8;
            ldsm_x4_t(vb, &Vt[Ring::off(vrow, np * 2 + (lane >> 4))]);
            mma_f16(o[2 * np], pa, vb[0], vb[1]);
            mma_f16(o[2 * np + 1], pa, vb[2], vb[3]);
        }
        ring.release(t);
    }
    ring.finish();
    // this item's partial (an empty split leaves max = -inf, sum = 0, which the merge ignores)
#pragma unroll
    for (int hf = 0; hf < 2; hf++) {
        float l = l_run[hf];
        l += __shfl_xor_sync(0xffffffffu, l, 1);
        l += __shfl_xor_sync(0xffffffffu, l, 2);
        const int qi = (lane >> 2) + hf * 8;
        if (qi < nq_here) {
            const int qg = q0 + qi, r = qg / G, j = qg % G;
            const size_t cell = ((size_t)(row0 + r) * a.Hq + hk * G + j) * splits + sp;
            if ((lane & 3) == 0) a.part_ml[cell] = make_float2(m_run[hf] * LN2, l);  // max back in natural-log units
#pragma unroll
            for (int nt = 0; nt < HD / 8; nt++)
                *reinterpret_cast<float2 *>(a.part_o + cell * HD + nt * 8 + (lane & 3) * 2) =
                    make_float2(o[nt][hf * 2], o[nt][hf * 2 + 1]);
        }
    }
}

// One item of at most eight query vectors, by one warp, in the transposed form: with few query
// heads per kv head (a single row of a group) the sixteen-row M dimension of the form above is
// half empty, so here the POSITIONS are the M dimension.  S^T = K Q^T (K tile as the A operand,
// the queries as eight B columns, 16 registers for the whole item), the softmax runs down the
// columns (maxima and sums across the eight lane groups), P^T becomes the B operand of
// O^T = V^T P^T through two 8x8 register transposes, and V^T is read with transposing ldmatrix.
// Half the MMAs, half the accumulators and a quarter of the exponentials of the other form;
// the partial it writes is the same.
template <int HD, int NS, bool TMA>
__device__ __forceinline__ void attn_item_t(const AttnArgs &a, const AtItem &it, kv_t *wr, int lane, AttnTma *tm = nullptr)
{
    constexpr float LOG2E = 1.4426950408889634f, LN2 = 0.6931471805599453f;
    typedef AtRing<HD, NS, TMA> Ring;
    const int G = a.Hq / a.Hkv, splits = a.n_splits;
    const int hk = it.hk, sp = it.sp, row0 = it.row0, pos0 = it.pos0;
    const int nq = it.nq;  // <= 8
    if (it.n_tiles == 0) {
        for (int qi = lane; qi < nq; qi += 32)
            a.part_ml[((size_t)(row0 + qi / G) * a.Hq + hk * G + qi % G) * splits + sp] = make_float2(-INFINITY, 0.f);
        return;
    }
    Ring ring(a, it, wr, lane, tm);
    ring.start();

    // the queries as B fragments: column lane / 4, elements 2 (lane % 4) + {0, 1, 8, 9} of every
    // 16-element step, scaled by log2(e) / sqrt(hd)
    uint32_t qf[HD / 16][2];
    {
        const int qi = lane >> 2, c0 = (lane & 3) * 2;
        const bool have = qi < nq;
        const size_t o = (size_t)(row0 + (have ? qi / G : 0)) * a.Hq * HD + (hk * G + (have ? qi % G : 0)) * HD + c0;
        const float qscale = rsqrtf((float)HD) * LOG2E;
#pragma unroll
        for (int ks = 0; ks < HD / 16; ks++) {
            float2 x0 = make_float2(0.f, 0.f), x1 = x0;
            if (have) {
                if (a.q32) {
                    x0 = *reinterpret_cast<const float2 *>(a.q32 + o + ks * 16);
                    x1 = *reinterpret_cast<const float2 *>(a.q32 + o + ks * 16 + 8);
                } else {
                    const uint32_t u0 = *reinterpret_cast<const uint32_t *>(a.q + o + ks * 16);
                    const uint32_t u1 = *reinterpret_cast<const uint32_t *>(a.q + o + ks * 16 + 8);
                    x0 = make_float2(bf_lo(u0), bf_hi(u0));
                    x1 = make_float2(bf_lo(u1), bf_hi(u1));
                }
            }
            qf[ks][0] = pack_h2(x0.x * qscale, x0.y * qscale);
            qf[ks][1] = pack_h2(x1.x * qscale, x1.y * qscale);
        }
    }
    // this thread's two query vectors (accumulator columns) and the last position each may see
    int limit[2];
#pragma unroll
    for (int e = 0; e < 2; e++) {
        const int qi = (lane & 3) * 2 + e;
        limit[e] = qi < nq ? pos0 + qi / G : -1;
    }
    float o[HD / 16][4], m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};
#pragma unroll
    for (int mt = 0; mt < HD / 16; mt++)
#pragma unroll
        for (int e = 0; e < 4; e++) o[mt][e] = 0.f;

    for (int t = 0; t < ring.n_tiles; t++) {
        const kv_t *Kt, *Vt;
        if (!ring.wait(t, Kt, Vt)) return;
        const int p0 = ring.w_beg + t * AT_TP;
        // S^T for 16 positions x 8 query vectors, two accumulator chains
        float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int ks = 0; ks < HD / 16; ks += 2) {
            uint32_t ka[4], kb[4];
            ldsm_x4(ka, &Kt[Ring::off(lane & 15, ks * 2 + (lane >> 4))]);
            ldsm_x4(kb, &Kt[Ring::off(lane & 15, (ks + 1) * 2 + (lane >> 4))]);
            mma_f16(s0, ka, qf[ks][0], qf[ks][1]);
            mma_f16(s1, kb, qf[ks + 1][0], qf[ks + 1][1]);
        }
        // online softmax down the columns; accumulator rows are positions lane / 4 and + 8
        const bool full = p0 + AT_TP <= ring.w_end && p0 + AT_TP - 1 <= pos0;
        float pv[2][2], alpha[2];
#pragma unroll
        for (int e = 0; e < 2; e++) {
#pragma unroll
            for (int j = 0; j < 2; j++) {
                const int p = p0 + (lane >> 2) + j * 8;
                const bool ok = full || (p < ring.w_end && p <= limit[e]);
                pv[e][j] = ok ? s0[j * 2 + e] + s1[j * 2 + e] : -INFINITY;
            }
            float tmax = fmaxf(pv[e][0], pv[e][1]);
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 4));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 8));
            tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 16));
            const float m_new = fmaxf(m_run[e], tmax);
            alpha[e] = 1.f;
            if (m_new != -INFINITY) {
                alpha[e] = exp2f(m_run[e] - m_new);
                pv[e][0] = exp2f(pv[e][0] - m_new);
                pv[e][1] = exp2f(pv[e][1] - m_new);
            } else {
                pv[e][0] = pv[e][1] = 0.f;
            }
            l_run[e] = l_run[e] * alpha[e] + pv[e][0] + pv[e][1];  // per-thread share; lanes are summed at the end
            m_run[e] = m_new;
        }
        // P^T as the B operand: the accumulator layout of an 8x8 block (row = position, two
        // columns = query vectors) transposed is the operand layout (row = query vector ...)
        const uint32_t b0 = movmatrix_t(pack_h2(pv[0][0], pv[1][0]));  // positions 0..7 of the tile
        const uint32_t b1 = movmatrix_t(pack_h2(pv[0][1], pv[1][1]));  // positions 8..15
        if (__any_sync(0xffffffffu, alpha[0] != 1.f || alpha[1] != 1.f)) {
#pragma unroll
            for (int mt = 0; mt < HD / 16; mt++) {
                o[mt][0] *= alpha[0];
                o[mt][1] *= alpha[1];
                o[mt][2] *= alpha[0];
                o[mt][3] *= alpha[1];
            }
        }
        // O^T += V^T P^T: sixteen dimensions per MMA, V read transposed
#pragma unroll
        for (int mt = 0; mt < HD / 16; mt++) {
            uint32_t va[4];
            ldsm_x4_t(va, &Vt[Ring::off((lane & 7) + ((lane >> 4) << 3), mt * 2 + ((lane >> 3) & 1))]);
            mma_f16(o[mt], va, b0, b1);
        }
        ring.release(t);
    }
    ring.finish();
#pragma unroll
    for (int e = 0; e < 2; e++) {
        float l = l_run[e];
        l += __shfl_xor_sync(0xffffffffu, l, 4);
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        const int qi = (lane & 3) * 2 + e;
        if (qi < nq) {
            const size_t cell = ((size_t)(row0 + qi / G) * a.Hq + hk * G + qi % G) * splits + sp;
            if ((lane >> 2) == 0) a.part_ml[cell] = make_float2(m_run[e] * LN2, l);
#pragma unroll
            for (int mt = 0; mt < HD / 16; mt++) {
                a.part_o[cell * HD + mt * 16 + (lane >> 2)] = o[mt][e];
                a.part_o[cell * HD + mt * 16 + 8 + (lane >> 2)] = o[mt][2 + e];
            }
        }
    }
}

// Persistent grid of warps; item i = ((sp * groups + g) * Hkv + hk) * n_qblk + qb: the query
// blocks of one (group, kv head, split) run side by side, and all but the first find their K/V
// tiles in the L2; the splits that short groups leave empty come last.  With a ticket counter
// the warps draw items as they finish (ragged lengths make the items of a round-robin deal
// uneven: a third of the warps idle on average at 64 sequences of 256..2048 positions);
// without one, item i goes to warp i mod (number of warps), warps numbered so that consecutive
// items land on different SMs.
template <int HD, int NST>
__global__ void __launch_bounds__(AW_WARPS * 32) attn_warp_kernel(AttnArgs a)
{
    extern __shared__ __align__(16) unsigned char aw_smem[];
    griddep_launch();
    griddep_wait();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    kv_t *wr = reinterpret_cast<kv_t *>(aw_smem) + (size_t)warp * NST * 2 * AT_TP * (HD + 8);
    const int n_groups = min(*a.n_groups, a.max_groups);
    const unsigned n_items = (unsigned)a.max_groups * a.n_qblk * a.Hkv * a.n_splits;
    const unsigned n_workers = gridDim.x * AW_WARPS;
    // every warp's first item is its own number (no counter, no latency); tickets number the
    // items beyond that first round, so a launch with no more items than warps draws none
    const bool dynamic = a.ticket != nullptr && n_items > n_workers;
    auto draw = [&]() -> unsigned {
        unsigned t = 0;
        if (lane == 0) t = atomicAdd(a.ticket, 1u) - a.ticket_base;
        return n_workers + __shfl_sync(0xffffffffu, t, 0);
    };
    unsigned item = (unsigned)warp * gridDim.x + blockIdx.x;
    while (item < n_items) {
        // the next ticket is drawn before this item's work, so that its latency is hidden
        const unsigned next = dynamic ? draw() : item + n_workers;
        const AtItem it = at_resolve(a, item, n_items, n_groups, a.grp_row0, a.grp_nrows, a.row_slot, a.row_pos);
        item = next;
        if (!it.valid) continue;
        if (it.nq <= 8) attn_item_t<HD, NST, false>(a, it, wr, lane);
        else attn_item<HD, NST, true>(a, it, wr, nullptr, lane);
    }
}

// The same grid with TMA-fed rings (callers that hold tensor maps of the cache: the decode
// path).  Without the padding and with one copy per tile a warp's stage is 16 positions x
// head_dim x 2 matrices x 2 bytes, so three CTAs per SM hold either four warps with two stages or
// three warps with three.
template <int HD, int NST, int WARPS>
__global__ void __launch_bounds__(WARPS * 32) attn_warp_tma_kernel(const __grid_constant__ CUtensorMap map_k,
                                                                      const __grid_constant__ CUtensorMap map_v, AttnArgs a,
                                                                      int *status)
{
    extern __shared__ __align__(1024) unsigned char awt_smem[];
    __shared__ __align__(8) uint64_t bars[WARPS][NST];
    __shared__ int giving_up_s;
    griddep_launch();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int w = 0; w < WARPS; w++)
            for (int s = 0; s < NST; s++) mbar_init(&bars[w][s], 1);
        giving_up_s = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    griddep_wait();
    // swizzled tiles want 1024-byte alignment
    unsigned char *ring = awt_smem + ((1024u - (smem_u32(awt_smem) & 1023u)) & 1023u);
    kv_t *wr = reinterpret_cast<kv_t *>(ring) + (size_t)warp * NST * 2 * AT_TP * HD;
    AttnTma tm;
    tm.mk = &map_k; tm.mv = &map_v; tm.bars = bars[warp]; tm.seq = 0; tm.giving_up = &giving_up_s; tm.status = status;
    const int n_groups = min(*a.n_groups, a.max_groups);
    const unsigned n_items = (unsigned)a.max_groups * a.n_qblk * a.Hkv * a.n_splits;
    const unsigned n_workers = gridDim.x * WARPS;
    const bool dynamic = a.ticket != nullptr && n_items > n_workers;
    auto draw = [&]() -> unsigned {
        unsigned t = 0;
        if (lane == 0) t = atomicAdd(a.ticket, 1u) - a.ticket_base;
        return n_workers + __shfl_sync(0xffffffffu, t, 0);
    };
    unsigned item = (unsigned)warp * gridDim.x + blockIdx.x;
    while (item < n_items) {
        const unsigned next = dynamic ? draw() : item + n_workers;
        const AtItem it = at_resolve(a, item, n_items, n_groups, a.grp_row0, a.grp_nrows, a.row_slot, a.row_pos);
        item = next;
        // after a wait that ran out the warp keeps drawing (the ticket count must come out) but works no more
        if (!it.valid || giving_up_s) continue;
        if (it.nq <= 8) attn_item_t<HD, NST, true>(a, it, wr, lane, &tm);
        else attn_item<HD, NST, true, true>(a, it, wr, nullptr, lane, &tm);
    }
}
inline size_t attn_warp_tma_bytes(int head_dim, int stages, int warps)
{
    return (size_t)warps * stages * 2 * AT_TP * head_dim * sizeof(kv_t) + 1024;
}
typedef void (*AttnWarpTmaFn)(const CUtensorMap, const CUtensorMap, AttnArgs, int *);
// The instantiation for a head dimension (64 or 128) and a ring depth (2: four warps per CTA,
// 3: three), its dynamic shared-memory limit raised on first use.
inline cudaError_t attn_warp_tma_fn(int head_dim, int stages, AttnWarpTmaFn *fn, int *warps)
{
    static PerDevice<bool> ready_dev[4];
    const int idx = (head_dim == 128 ? 2 : 0) + (stages == 3 ? 1 : 0);
    AttnWarpTmaFn f = idx == 3 ? attn_warp_tma_kernel<128, 3, 3> : idx == 2 ? attn_warp_tma_kernel<128, 2, 4>
                      : idx == 1 ? attn_warp_tma_kernel<64, 3, 3> : attn_warp_tma_kernel<64, 2, 4>;
    *warps = stages == 3 ? 3 : 4;
    bool &ready = ready_dev[idx].here();
    if (!ready) {
        const cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)attn_warp_tma_bytes(head_dim, stages, *warps));
        if (e != cudaSuccess) return e;
        ready = true;
    }
    *fn = f;
    return cudaSuccess;
}

// The grid of the stand-alone kernel: as many CTAs as fit the SMs (registers allow three).
inline int attn_warp_ctas_per_sm(int head_dim, int stages)
{
    const size_t per_cta = AW_WARPS * attn_warp_bytes(head_dim, stages) + 1024;
    const int by_smem = (int)((size_t)227 * 1024 / per_cta);
    return by_smem < 1 ? 1 : (by_smem > 3 ? 3 : by_smem);
}
typedef void (*AttnWarpFn)(AttnArgs);
// The instantiation for a head dimension (64 or 128) and a ring depth (2 or 3), its dynamic
// shared-memory limit raised on first use.
inline cudaError_t attn_warp_fn(int head_dim, int stages, AttnWarpFn *fn)
{
    static PerDevice<bool> ready_dev[4];
    const int idx = (head_dim == 128 ? 2 : 0) + (stages == 3 ? 1 : 0);
    AttnWarpFn f = idx == 3 ? attn_warp_kernel<128, 3> : idx == 2 ? attn_warp_kernel<128, 2>
                   : idx == 1 ? attn_warp_kernel<64, 3> : attn_warp_kernel<64, 2>;
    bool &ready = ready_dev[idx].here();
    if (!ready) {
        const cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                                   (int)(AW_WARPS * attn_warp_bytes(head_dim, stages)));
        if (e != cudaSuccess) return e;
        ready = true;
    }
    *fn = f;
    return cudaSuccess;
}

// Merge the splits of every (row, query head): out = sum_s acc_s e^{m_s - M} / sum_s l_s e^{m_s - M}.
// One block per (row, head), one thread per output dimension.  The splits' weights are worked out
// once (thread s takes split s) and parked in shared memory, so that the loop over the splits is
// a row of independent loads and not a chain of (max, sum) look-ups in front of every one.
template <int HD>
__global__ void __launch_bounds__(HD) attn_merge_kernel(AttnArgs a, const int *__restrict__ n_rows)
{
    __shared__ float w_s[AT_MAX_SPLITS];
    __shared__ float den_s;
    griddep_launch();
    griddep_wait();
    const int row = blockIdx.x, head = blockIdx.y;
    if (row >= *n_rows) return;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const size_t cell0 = ((size_t)row * a.Hq + head) * a.n_splits;
    // a.n_splits <= AT_MAX_SPLITS = 32 <= HD: the first warp holds one split per lane
    float2 ml = make_float2(-INFINITY, 0.f);
    if (tid < a.n_splits) ml = a.part_ml[cell0 + tid];
    if (warp == 0) {
        const float M = warp_max(ml.x);
        const float w = ml.x == -INFINITY ? 0.f : __expf(ml.x - M);
        const float den = warp_sum(ml.y * w);
        if (lane < AT_MAX_SPLITS) w_s[lane] = w;
        if (lane == 0) den_s = den;
    }
    __syncthreads();
    const float den = den_s;
    float num = 0.f;
#pragma unroll 4
    for (int s = 0; s < a.n_splits; s++) {
        const float w = w_s[s];
        if (w != 0.f) num += a.part_o[(cell0 + s) * HD + tid] * w;  // an empty split's partial is never read
    }
    const float val = den > 0.f ? num / den : 0.f;
    const bf16 hi = __float2bfloat16(val);
    a.out[(size_t)row * a.Hq * HD + head * HD + tid] = hi;
    if (a.out_lo) a.out_lo[(size_t)row * a.Hq * HD + head * HD + tid] = __float2bfloat16(val - __bfloat162float(hi));
}

}  // namespace sparsk

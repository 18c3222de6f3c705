// Host side of the SPAR-K decode library: argument checks, the host mirror of the exit
// schedule (which only sizes launches; the device kernels are authoritative), workspace
// carving and the launch sequence of a step.  C ABI declared in include/sparsk.h.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <vector>

#include "../../include/sparsk.h"
#include "sparsk_attn.cuh"
#include "sparsk_attn_tc.cuh"
#include "sparsk_common.cuh"
#include "sparsk_gemm.cuh"
#include "sparsk_gemv.cuh"
#include "sparsk_mega.cuh"
#include "sparsk_sample.cuh"
#include "sparsk_step.cuh"

using namespace sparsk;

namespace {

constexpr int MAX_SPLITS = AT_MAX_SPLITS;
constexpr int STAGE_RING = 16;
constexpr uint32_t CTX_MAGIC = 0x5350524bu;  // "SPRK"
constexpr size_t TIME_POOL = 16384;           // event pairs available to the kernel timer
enum { KC_MISC = 0, KC_QKV = 1, KC_ATTN = 2, KC_OPROJ = 3, KC_GATEUP = 4, KC_DOWN = 5, KC_HEAD = 6, KC_MEGA = 7, KC_ALL = 8 };

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Carve {
    char *base;
    size_t off;
    template <class T>
    T *take(size_t n)
    {
        off = align_up(off, 256);
        T *p = base ? reinterpret_cast<T *>(base + off) : nullptr;
        off += n * sizeof(T);
        return p;
    }
};

}  // namespace

struct TmaPair {
    CUtensorMap m2, m3;
};

struct sparsk_ctx {
    uint32_t magic;
    sparsk_dims dm;
    std::vector<const bf16 *> attn_norm, wq, wk, wv, wo, mlp_norm, w_gate, w_up, w_down, head_norm, head_proj;
    const bf16 *embed;
    cudaStream_t stream;
    int n_sm;
    int cap_rows;  // rows any pass may have
    // workspace
    kv_t *kcache, *vcache;
    float *pend_h;
    int *kv_len, *pend_cnt;
    float2 *rope;
    StepDesc sd;
    int *staged, *tok_dev, *out_tok_dev, *out_depth_dev;
    int *pf_slot, *pf_pos, *pf_grp_row0, *pf_grp_nrows, *pf_ngrp, *pf_nrows;
    float *h_lo, *h_up;
    float *qbuf;
    float *h_last, *q_last;      // the current rows alone, for the trimmed last layer of the upper pass
    int *last_slot, *last_pos;
    int trim_last;               // 0: never, 1: when it pays (default), 2: whenever there are pending rows
    bf16 *attn_o, *act, *xnorm;
    bf16 *attn_o_lo, *act_lo, *xnorm_lo;  // second bf16 term of the tensor-core path's activations
    float *part_o;
    float2 *part_ml;
    unsigned *attn_ticket;       // device: item counter of the attention kernel (only ever grows)
    unsigned attn_ticket_base;   // host: its value once every launch so far has finished
    int attn_dynamic;            // option: deal attention items by ticket (1, default) or round-robin (0)
    int attn_ctas;               // option: CTAs of the attention kernel (0: as many as fit the SMs)
    // pinned staging ring for the per-step host arrays
    int *stage_host[STAGE_RING];
    int *io_host;                // pinned: [B] tokens in, [B] tokens out, [B] depths out, status (decode_step_host)
    cudaEvent_t stage_ev[STAGE_RING];
    int stage_next;
    // host mirror of per-slot state
    std::vector<int> h_len, h_pend;
    // options
    int pdl, attn_split, gemm_min_rows, gv_ks, gv_r;
    float *dbg_hidden, *dbg_logits;
    // nucleus sampling (off while samp_uniforms is NULL)
    float samp_temperature, samp_top_p;
    const float *samp_uniforms;  // device [max_seqs], read by every decode step
    float *samp_scratch;         // device [max_seqs][Vt + Vs]
    int64_t launches;
    // tensor-core path: TMA descriptors of every weight matrix and of the activation buffers
    // (one per box height 16, 32, 64, 128, 256)
    bool tc_ok;
    std::vector<TmaPair> tm_wq, tm_wk, tm_wv, tm_wo, tm_wg, tm_wu, tm_wd, tm_head;
    TmaPair tm_x[5], tm_ao[5], tm_act[5], tm_x_lo[5], tm_ao_lo[5], tm_act_lo[5];
    std::vector<CUtensorMap> tm_kc16, tm_vc16;  // per layer: the cache as rows of head_dim numbers, boxes of 16 rows (attn_warp_tma_kernel)
    int attn_tma, attn_tma_ok;               // option (default 1); the maps above exist
    std::vector<CUtensorMap> tm_kc, tm_vc;  // per layer: the cache viewed as [64][slots * Hkv * S rows][hd / 64], boxes of [64][64][2]
    int attn_stages;                        // K/V ring depth of the warp-per-item attention kernel (2 or 3)
    int attn_tc, attn_tc_min_q;             // tcgen05 attention for blocks of at least this many query vectors
    // persistent layer-range kernel (one or two rows)
    MkLayer *mk_layers;            // device [L]
    unsigned long long *mk_bar;    // device: grid barrier counter; mk_bar_base mirrors its value
    int *mk_abort;                 // device
    float *mk_attn_o, *mk_act;     // device fp32 [MK_MAX_ROWS][Hq*hd], [MK_MAX_ROWS][F]
    unsigned long long *mk_trace;  // device [1 + 6 L]
    int mk_trace_n;                // entries the last launch wrote
    unsigned long long mk_bar_base;
    int mega, mk_ok, mk_coop, mk_max_rows;
    bool mk_tc_ok;                 // the shape allows the persistent kernel's tensor-core form (3-4 rows)
    // confidence-based exit (dims.conf_modalities != 0): the host drives the step layer by layer
    std::vector<std::vector<int>> h_fill;  // per slot: layer each pending position has been carried to
    int *conf_host;                // pinned arena for the row sets of a step's segments
    size_t conf_host_ints, conf_seg_ints;
    int *conf_rows_dev;            // device: [slot R][pos R][src R][seq R][grp_row0 B][grp_nrows B][n_groups][n_rows]
    int *conf_list_dev;            // device: [rows B][modality B]
    float *conf_ent_dev, *conf_ent_host;  // entropies of a layer's candidates (device, pinned host)
    std::vector<float> conf_trace; // last step: entropy seen at layer l (1-based, < L) by sequence i at [i * L + l], or -1
    float *conf_logits;            // device [B][V] when neither the parity hook nor a sampler lends a buffer
    int inject_timeout;            // test hook: the next persistent launch waits for a barrier count nobody reaches
    int64_t route_layers[3];       // layer passes so far by implementation: see sparsk_route_counts
    std::vector<MkLayer> mk_host;
    float *qkv_part;  // fp32 sums of a q/k/v product whose inner dimension is cut across CTAs
    int tc_kb;        // 0: automatic; 1: force one k-block per copy (2-D descriptors)
    int gemm_smem_kb; // shared-memory budget of a tcgen05 GEMM CTA
    int gemm_cps;     // CTAs per SM a split GEMM is cut for (1 or 2; 2 needs a budget that lets two share an SM)
    // optional per-kernel-class timing (events around every launch of one class)
    int cur_class, time_class;
    std::vector<cudaEvent_t> tev;
    std::vector<unsigned char> tev_class;  // class of each bracketed launch
    size_t tev_used;
    char err[512];
};

namespace {

int fail(sparsk_ctx *c, int code, const char *fmt, ...)
{
    if (c) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(c->err, sizeof c->err, fmt, ap);
        va_end(ap);
    }
    return code;
}

#define CU(call)                                                                                   \
    do {                                                                                           \
        cudaError_t e_ = (call);                                                                   \
        if (e_ != cudaSuccess)                                                                     \
            return fail(ctx, SPARSK_ECUDA, "%s failed: %s (%s:%d)", #call, cudaGetErrorString(e_), \
                        __FILE__, __LINE__);                                                       \
    } while (0)

bool dims_ok(const sparsk_dims *d)
{
    if (!d) return false;
    if (d->n_layers < 1 || d->d_model < 8 || d->d_model % 8) return false;
    if (d->n_q_heads < 1 || d->n_kv_heads < 1 || d->n_q_heads % d->n_kv_heads) return false;
    if (d->head_dim != 64 && d->head_dim != 128) return false;
    if (d->d_ffn < 8 || d->d_ffn % 8) return false;
    if (d->vocab_text < 1 || d->vocab_speech < 0) return false;
    if (!(d->rms_eps >= 0.f) || !(d->rope_base > 0.f)) return false;
    if (d->exit_layer < 1 || d->exit_layer > d->n_layers) return false;
    if (d->refresh_period < 1 || d->refresh_phase < 0 || d->refresh_phase >= d->refresh_period) return false;
    if (d->text_exit < 0 || d->text_exit > 2) return false;
    if (d->conf_modalities < 0 || d->conf_modalities > 3) return false;
    if (d->conf_modalities && (d->conf_start < 1 || d->conf_start >= d->n_layers || !(d->conf_threshold >= 0.f))) return false;
    if (d->text_period < 0 || (d->text_period > 0 && (d->text_phase < 0 || d->text_phase >= d->text_period))) return false;
    if (d->max_seqs < 1 || d->max_seqs > 1024 || d->max_seq_len < 1) return false;
    if (d->max_pending < 0 || d->prefill_rows < 0) return false;
    return true;
}

int cap_rows_of(const sparsk_dims *d)
{
    const int pf = d->prefill_rows > 0 ? d->prefill_rows : 64;
    const long dec = (long)d->max_seqs * (d->max_pending + 1);
    return (int)std::max<long>(dec, pf);
}

// Lays the workspace out; with base == NULL only measures it.
size_t carve(sparsk_ctx *c, const sparsk_dims *d, char *base)
{
    Carve w{base, 0};
    const size_t B = d->max_seqs, S = d->max_seq_len, L = d->n_layers;
    const size_t kvrow = (size_t)d->n_kv_heads * d->head_dim, qrow = (size_t)d->n_q_heads * d->head_dim;
    const size_t R = cap_rows_of(d);
    kv_t *kc = w.take<kv_t>(L * B * S * kvrow);
    kv_t *vc = w.take<kv_t>(L * B * S * kvrow);
    float *ph = w.take<float>(B * (size_t)std::max(1, d->max_pending) * d->d_model);
    int *kl = w.take<int>(B), *pc = w.take<int>(B);
    float2 *rope = w.take<float2>(S * (d->head_dim / 2));
    StepDesc sd;
    sd.slot = w.take<int>(B); sd.modality = w.take<int>(B); sd.counter = w.take<int>(B);
    sd.token = w.take<int>(B); sd.depth = w.take<int>(B); sd.lo_pos = w.take<int>(B);
    sd.lo_grp_row0 = w.take<int>(B); sd.lo_grp_nrows = w.take<int>(B);
    sd.up_slot = w.take<int>(R); sd.up_pos = w.take<int>(R); sd.up_src = w.take<int>(R);
    sd.up_grp_row0 = w.take<int>(B); sd.up_grp_nrows = w.take<int>(B); sd.cur_row = w.take<int>(B);
    sd.list_seq = w.take<int>(4 * B); sd.list_row = w.take<int>(4 * B);
    sd.counts = w.take<int>(8);
    sd.argmax = w.take<unsigned long long>(B);
    int *staged = w.take<int>(3 * B), *tok = w.take<int>(B), *ot = w.take<int>(B), *od = w.take<int>(B);
    int *pfs = w.take<int>(R), *pfp = w.take<int>(R), *pfg0 = w.take<int>(1), *pfgn = w.take<int>(1);
    int *pfng = w.take<int>(1), *pfnr = w.take<int>(1);
    float *hlo = w.take<float>(B * d->d_model), *hup = w.take<float>(R * d->d_model);
    float *q = w.take<float>(R * qrow);
    int *crows = nullptr, *clist = nullptr;
    float *cent = nullptr, *clog = nullptr;
    if (d->conf_modalities) {
        crows = w.take<int>(4 * R + 2 * B + 2);
        clist = w.take<int>(2 * B);
        cent = w.take<float>(B);
        clog = w.take<float>(B * ((size_t)d->vocab_text + d->vocab_speech));
    }
    float *hlast = w.take<float>(B * d->d_model), *qlast = w.take<float>(B * qrow);
    int *lslot = w.take<int>(B), *lpos = w.take<int>(B);
    bf16 *ao = w.take<bf16>(R * qrow), *act = w.take<bf16>(R * d->d_ffn);
    bf16 *xn = w.take<bf16>(R * d->d_model);
    bf16 *aol = w.take<bf16>(R * qrow), *actl = w.take<bf16>(R * d->d_ffn), *xnl = w.take<bf16>(R * d->d_model);
    float *qp = w.take<float>(R * (qrow + 2 * kvrow));
    MkLayer *mkl = w.take<MkLayer>(L);
    unsigned long long *mkb = w.take<unsigned long long>(1);
    int *mka = w.take<int>(1);
    unsigned *atk = w.take<unsigned>(1);
    float *mkao = w.take<float>((size_t)MK_MAX_ROWS * qrow), *mkact = w.take<float>((size_t)MK_MAX_ROWS * d->d_ffn);
    unsigned long long *mkt = w.take<unsigned long long>(1 + 6 * L);
    const size_t cells = std::max<size_t>(R * MAX_SPLITS, (size_t)MK_MAX_ROWS * MK_MAX_SPLITS) * d->n_q_heads;
    float *po = w.take<float>(cells * d->head_dim);
    float2 *pml = w.take<float2>(cells);
    if (c) {
        c->kcache = kc; c->vcache = vc; c->pend_h = ph; c->kv_len = kl; c->pend_cnt = pc; c->rope = rope;
        c->sd = sd; c->staged = staged; c->tok_dev = tok; c->out_tok_dev = ot; c->out_depth_dev = od;
        c->pf_slot = pfs; c->pf_pos = pfp; c->pf_grp_row0 = pfg0; c->pf_grp_nrows = pfgn;
        c->pf_ngrp = pfng; c->pf_nrows = pfnr;
        c->conf_rows_dev = crows; c->conf_list_dev = clist; c->conf_ent_dev = cent; c->conf_logits = clog;
        c->h_last = hlast; c->q_last = qlast; c->last_slot = lslot; c->last_pos = lpos;
        c->h_lo = hlo; c->h_up = hup; c->qbuf = q; c->attn_o = ao; c->act = act; c->xnorm = xn; c->qkv_part = qp;
        c->attn_o_lo = aol; c->act_lo = actl; c->xnorm_lo = xnl;
        c->mk_layers = mkl; c->mk_bar = mkb; c->mk_abort = mka; c->mk_attn_o = mkao; c->mk_act = mkact; c->mk_trace = mkt;
        c->part_o = po; c->part_ml = pml; c->attn_ticket = atk;
    }
    return align_up(w.off, 256);
}

template <class... KArgs, class... Args>
cudaError_t launch(sparsk_ctx *c, void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, Args... args)
{
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute attr[1];
    if (c->pdl) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
    }
    c->launches++;
    const bool timed = ((c->time_class == c->cur_class && c->time_class != KC_MISC) || c->time_class == KC_ALL) &&
                       c->tev_used + 2 <= c->tev.size();
    if (timed) {
        c->tev_class[c->tev_used / 2] = (unsigned char)c->cur_class;
        cudaEventRecord(c->tev[c->tev_used++], c->stream);
    }
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, KArgs(args)...);
    if (timed) cudaEventRecord(c->tev[c->tev_used++], c->stream);
    return e;
}

// ---------------------------------------------------------------- GEMV dispatch
struct GvPlan {
    int ks, grid_x;
};

GvPlan plan_gemv(const sparsk_ctx *c, int n_groups, int K)
{
    const int chunks = (K + 255) / 256;
    int best_ks = 1;
    double best = 1e30;
    for (int ks = 1; ks <= GV_WARPS; ks *= 2) {
        if (ks > 1 && ks > chunks) break;
        const long T = (long)c->n_sm * (GV_WARPS / ks);
        const long iters = (n_groups + T - 1) / T;
        const double cost = (double)iters * ((chunks + ks - 1) / ks + 3.0);
        if (cost < best - 1e-9) {
            best = cost;
            best_ks = ks;
        }
    }
    if (c->gv_ks > 0) best_ks = c->gv_ks;
    GvPlan p;
    p.ks = best_ks;
    p.grid_x = std::min(c->n_sm, n_groups);
    if (p.grid_x < 1) p.grid_x = 1;
    return p;
}

template <class Op, int R, int M, bool NORM>
cudaError_t launch_gemv_inst(sparsk_ctx *c, const Op &op, GvIn in, int n_groups)
{
    static PerDevice<bool> attr_done;
    bool &attr_set = attr_done.here();
    auto kern = gemv_kernel<Op, R, M, NORM>;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const GvPlan p = plan_gemv(c, n_groups, in.K);
    in.ks = p.ks;
    const size_t smem = align_up((size_t)M * in.K * 2, 16) + (size_t)2 * GV_WARPS * R * M * sizeof(float);
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    const int passes = (M == GV_MC) ? (in.n_rows + GV_MC - 1) / GV_MC : 1;
    return launch(c, kern, dim3(p.grid_x, passes), dim3(GV_THREADS), smem, op, in);
}

// M template: 1, 2 or 4 (three rows run as four with one masked).
#define GV_DISPATCH_M(OPT, RR, NORM, op, in, ng)                                    \
    ((in).n_rows == 1   ? launch_gemv_inst<OPT<RR>, RR, 1, NORM>(c, op, in, ng)     \
     : (in).n_rows == 2 ? launch_gemv_inst<OPT<RR>, RR, 2, NORM>(c, op, in, ng)     \
                        : launch_gemv_inst<OPT<RR>, RR, 4, NORM>(c, op, in, ng))

int pick_r(const sparsk_ctx *c, int n_rows, bool paired)
{
    if (c->gv_r > 0) return (paired && c->gv_r < 2) ? 2 : c->gv_r;
    if (n_rows >= 3) return 4;
    return 2;
}

struct RowSet {
    const int *slot, *pos, *grp_row0, *grp_nrows, *n_groups, *n_rows_dev;
    int n_rows;     // host count (sizes the launches)
    int n_groups_h; // host count
    int max_grp_rows;
    int max_len;    // longest prefix any row attends to (host)
    int n_big;      // groups with at least attn_tc_min_q query vectors per kv head (0: not counted, assume all)
    const float *q; // the rows' queries if they are not the context's query buffer (NULL: they are)
    long sum_len;   // total of the groups' prefix lengths (host; 0: unknown)
};

cudaError_t run_qkv(sparsk_ctx *c, int layer, const float *h, const RowSet &rs)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1;
    GvIn in{};
    in.h = h; in.gain = c->attn_norm[li]; in.eps = d.rms_eps; in.K = d.d_model; in.n_rows = rs.n_rows;
    const size_t lstride = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len * d.head_dim;
    const int R = pick_r(c, rs.n_rows, true);
#define QKV_CASE(RR)                                                                                   \
    {                                                                                                  \
        QkvOp<RR> op;                                                                                  \
        op.wq = c->wq[li]; op.wk = c->wk[li]; op.wv = c->wv[li]; op.q_out = c->qbuf;                   \
        op.kc = c->kcache + li * lstride; op.vc = c->vcache + li * lstride; op.rope = c->rope;         \
        op.row_slot = rs.slot; op.row_pos = rs.pos; op.d = d.d_model; op.Hq = d.n_q_heads;             \
        op.Hkv = d.n_kv_heads; op.hd = d.head_dim; op.S = d.max_seq_len;                               \
        const int P = RR / 2;                                                                          \
        const int ng = (d.n_q_heads + d.n_kv_heads) * (d.head_dim / 2) / P + d.n_kv_heads * d.head_dim / RR; \
        return GV_DISPATCH_M(QkvOp, RR, true, op, in, ng);                                             \
    }
    if (R == 4) QKV_CASE(4) else QKV_CASE(2)
#undef QKV_CASE
}

cudaError_t run_resid(sparsk_ctx *c, const bf16 *w, const bf16 *x, float *h, int K, int n_out, int n_rows)
{
    GvIn in{};
    in.x = x; in.K = K; in.n_rows = n_rows;
    int R = c->gv_r > 0 ? c->gv_r : (n_rows >= 3 ? 4 : 2);
#define RES_CASE(RR)                                            \
    {                                                           \
        ResidOp<RR> op;                                         \
        op.w = w; op.h = h; op.K = K; op.n_out = n_out;         \
        const int ng = (n_out + RR - 1) / RR;                   \
        return GV_DISPATCH_M(ResidOp, RR, false, op, in, ng);   \
    }
    if (R == 4) RES_CASE(4) else if (R == 2) RES_CASE(2) else RES_CASE(1)
#undef RES_CASE
}

cudaError_t run_gateup(sparsk_ctx *c, int layer, const float *h, int n_rows)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1;
    GvIn in{};
    in.h = h; in.gain = c->mlp_norm[li]; in.eps = d.rms_eps; in.K = d.d_model; in.n_rows = n_rows;
    const int R = pick_r(c, n_rows, true);
#define GU_CASE(RR)                                                              \
    {                                                                            \
        GateUpOp<RR> op;                                                         \
        op.wg = c->w_gate[li]; op.wu = c->w_up[li]; op.u = c->act;               \
        op.d = d.d_model; op.F = d.d_ffn;                                        \
        const int P = RR / 2;                                                    \
        const int ng = (d.d_ffn + P - 1) / P;                                    \
        return GV_DISPATCH_M(GateUpOp, RR, true, op, in, ng);                    \
    }
    if (R == 4) GU_CASE(4) else GU_CASE(2)
#undef GU_CASE
}

// Where the heads leave their logits: the parity hook's buffer, else the sampler's, else nowhere.
float *head_logits(const sparsk_ctx *c)
{
    return c->dbg_logits ? c->dbg_logits : (c->samp_uniforms ? c->samp_scratch : c->conf_logits);
}

bool use_tc(const sparsk_ctx *c, int n_rows);
cudaError_t run_head_tc(sparsk_ctx *c, int layer, const float *h, int list, int n_rows);

// Head of `layer` over list `l` (0 early/text, 1 early/speech, 2 full/text, 3 full/speech).
cudaError_t run_head(sparsk_ctx *c, int layer, const float *h, int list, int n_rows)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1, B = d.max_seqs;
    GvIn in{};
    in.h = h; in.gain = c->head_norm[li]; in.eps = d.rms_eps; in.K = d.d_model; in.n_rows = n_rows;
    in.row_idx = c->sd.list_row + (size_t)list * B;
    const int speech = list & 1;
    if (use_tc(c, n_rows)) return run_head_tc(c, layer, h, list, n_rows);
    const int R = c->gv_r > 0 ? c->gv_r : 4;
    struct ClassScope {
        sparsk_ctx *c;
        ~ClassScope() { c->cur_class = KC_MISC; }
    } scope{c};
    c->cur_class = KC_HEAD;
#define HD_CASE(RR)                                                                              \
    {                                                                                            \
        HeadOp<RR> op;                                                                           \
        op.w = c->head_proj[li]; op.seq_of_row = c->sd.list_seq + (size_t)list * B;              \
        op.argmax = c->sd.argmax; op.logits = head_logits(c); op.d = d.d_model;                   \
        op.lo = speech ? d.vocab_text : 0; op.hi = speech ? d.vocab_text + d.vocab_speech : d.vocab_text; \
        op.V = d.vocab_text + d.vocab_speech;                                                    \
        const int ng = (op.hi - op.lo + RR - 1) / RR;                                            \
        return GV_DISPATCH_M(HeadOp, RR, true, op, in, ng);                                      \
    }
    if (R == 4) HD_CASE(4) else if (R == 2) HD_CASE(2) else HD_CASE(1)
#undef HD_CASE
}

int div_up(int a, int b);

cudaError_t run_attn(sparsk_ctx *c, int layer, const RowSet &rs)
{
    const sparsk_dims &d = c->dm;
    const int G = d.n_q_heads / d.n_kv_heads;
    const size_t lstride = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len * d.head_dim;
    AttnArgs a{};
    a.q = nullptr;
    a.q32 = rs.q ? rs.q : c->qbuf;
    a.kc = c->kcache + (layer - 1) * lstride;
    a.vc = c->vcache + (layer - 1) * lstride;
    a.grp_row0 = rs.grp_row0; a.grp_nrows = rs.grp_nrows; a.row_slot = rs.slot; a.row_pos = rs.pos;
    a.n_groups = rs.n_groups;
    a.part_o = c->part_o; a.part_ml = c->part_ml; a.out = c->attn_o; a.out_lo = c->attn_o_lo;
    a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.S = d.max_seq_len;
    a.n_slots = d.max_seqs;
    a.n_rows = rs.n_rows;
    a.nq_min = 0;
    a.nq_max = 1 << 30;
    cudaError_t e;
    const bool blocks_tc = c->attn_tc && c->tc_ok && d.head_dim == TA_HD && rs.max_grp_rows * G >= c->attn_tc_min_q;
    // groups the tcgen05 kernel takes (the host knows every group's row count) and the rest
    const int n_big = blocks_tc ? (rs.n_big > 0 ? rs.n_big : rs.n_groups_h) : 0;
    const int n_small = rs.n_groups_h - n_big;
    const int warp_ctas = c->attn_ctas > 0 ? c->attn_ctas : c->n_sm * attn_warp_ctas_per_sm(d.head_dim, c->attn_stages);
    const int small_rows = blocks_tc ? std::max(1, std::min(rs.max_grp_rows, (c->attn_tc_min_q - 1) / G)) : rs.max_grp_rows;
    AttnPlan pl = attn_plan(warp_ctas * AW_WARPS, blocks_tc ? std::max(1, n_small) : rs.n_groups_h, small_rows, G,
                            d.n_kv_heads, rs.max_len, c->attn_split, blocks_tc ? 0 : rs.sum_len);
    if (blocks_tc) {
        // Groups with many query vectors per kv head go to the tcgen05 kernel (one CTA per SM, tiles
        // of 64 positions), the others to the mma.sync kernel; both launches cover all groups, a CTA
        // leaves at once if its group belongs to the other, and both use one split plan so that the
        // merge finds every partial where it expects it.
        static PerDevice<bool> ready_dev;
        bool &ready = ready_dev.here();
        if (!ready) {
            if ((e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TA_SMEM)) != cudaSuccess) return e;
            ready = true;
        }
        // The tcgen05 kernel wants few, long splits (about one CTA per SM from the big groups alone,
        // its set-up is worth a few tiles), the other kernel many short ones: the first kernel's
        // split is `mult` of the second's, and it marks the partial slots in between as empty.
        const int big_ctas = std::max(1, n_big * div_up(rs.max_grp_rows * G, TA_QB) * d.n_kv_heads);
        const int tiles = std::max(1, div_up(rs.max_len, TA_NT));
        int s_tc = 1;
        {   // the split count whose CTAs fill whole waves of one CTA per SM best (at least 8 tiles each)
            double best = -1.0;
            const int s_max = std::max(1, std::min(AT_MAX_SPLITS, tiles / 8));
            for (int sc = 1; sc <= s_max; sc++) {
                const long n = (long)big_ctas * sc, waves = (n + c->n_sm - 1) / c->n_sm;
                const double eff = (double)n / (double)(waves * c->n_sm);
                const double score = eff * (waves >= 2 ? 1.0 : 0.9);  // a second wave evens out ragged lengths
                if (score > best + 1e-9) {
                    best = score;
                    s_tc = sc;
                }
                if (waves >= 2 && eff >= 0.9) break;
            }
        }
        if (c->attn_split > 0) s_tc = pl.n_splits;
        s_tc = std::min(s_tc, AT_MAX_SPLITS);
        const int mult = std::max(1, std::min(AT_MAX_SPLITS / s_tc, div_up(pl.n_splits, s_tc)));
        const int small_len = div_up(div_up(rs.max_len, s_tc * mult), TA_NT) * TA_NT;
        pl.split_len = small_len;
        pl.n_splits = std::max(1, div_up(rs.max_len, small_len));
        AttnTcArgs ta;
        ta.a = a;
        ta.a.n_qblk = div_up(rs.max_grp_rows * G, TA_QB);
        ta.a.split_len = small_len * mult;
        ta.a.n_splits = pl.n_splits;
        ta.a.nq_min = c->attn_tc_min_q;
        ta.split_mult = mult;
        ta.status = c->sd.counts + CNT_STATUS;
        const int n_splits_tc = std::max(1, div_up(rs.max_len, small_len * mult));
        dim3 grid(rs.n_groups_h * ta.a.n_qblk, d.n_kv_heads, n_splits_tc);
        e = launch(c, attn_tc_kernel, grid, dim3(TA_THREADS), (size_t)TA_SMEM, c->tm_kc[layer - 1], c->tm_vc[layer - 1], ta);
        if (e != cudaSuccess) return e;
        a.nq_max = c->attn_tc_min_q - 1;
    }
    a.n_qblk = blocks_tc ? div_up(std::min(rs.max_grp_rows * G, c->attn_tc_min_q - 1), 16) : pl.n_qblk;
    a.split_len = pl.split_len;
    a.n_splits = pl.n_splits;
    a.max_groups = rs.n_groups_h;
    if (!blocks_tc || (c->attn_tc_min_q > 1 && n_small > 0)) {
        // every group is in the item space (the kernel skips those the other kernel takes)
        const long n_items = (long)rs.n_groups_h * a.n_qblk * d.n_kv_heads * a.n_splits;
        const bool tma = c->attn_tma && c->attn_tma_ok;
        int warps = AW_WARPS;
        AttnWarpFn fn = nullptr;
        AttnWarpTmaFn fn_tma = nullptr;
        e = tma ? attn_warp_tma_fn(d.head_dim, c->attn_stages, &fn_tma, &warps) : attn_warp_fn(d.head_dim, c->attn_stages, &fn);
        if (e != cudaSuccess) return e;
        const int grid = (int)std::max<long>(1, std::min<long>(warp_ctas, (n_items + warps - 1) / warps));
        if (c->attn_dynamic && n_items < (1L << 31)) {
            a.ticket = c->attn_ticket;
            a.ticket_base = c->attn_ticket_base;
        }
        if (tma)
            e = launch(c, fn_tma, dim3(grid), dim3(warps * 32), attn_warp_tma_bytes(d.head_dim, c->attn_stages, warps),
                       c->tm_kc16[layer - 1], c->tm_vc16[layer - 1], a, c->sd.counts + CNT_STATUS);
        else
            e = launch(c, fn, dim3(grid), dim3(warps * 32), AW_WARPS * attn_warp_bytes(d.head_dim, c->attn_stages), a);
        if (e != cudaSuccess) return e;
        // the items beyond the warps' first ones are drawn once each, and every warp draws one
        // ticket beyond its last item
        if (a.ticket && n_items > (long)grid * warps) c->attn_ticket_base += (unsigned)n_items;
    }
    if (d.head_dim == 128) return launch(c, attn_merge_kernel<128>, dim3(rs.n_rows, d.n_q_heads), dim3(128), 0, a, rs.n_rows_dev);
    return launch(c, attn_merge_kernel<64>, dim3(rs.n_rows, d.n_q_heads), dim3(64), 0, a, rs.n_rows_dev);
}

// ---------------------------------------------------------------- tensor-core dispatch
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Descriptors of a row-major bf16 matrix [rows][cols], 128-byte swizzle, zero fill outside:
// m2 reads boxes of [box_rows][64]; m3 (only when cols is a multiple of 64) views the matrix as
// [64][rows][cols/64] and reads [box_rows] rows of two consecutive 64-element blocks at once.
bool encode_maps(EncodeTiledFn fn, TmaPair *m, const void *base, size_t rows, size_t cols, int box_rows,
                 CUtensorMapDataType dtype = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16)
{
    memset(m, 0, sizeof *m);
    if (!base) return true;
    const cuuint32_t es[3] = {1, 1, 1};
    {
        const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
        const cuuint32_t box[2] = {(cuuint32_t)GM_BK, (cuuint32_t)box_rows};
        if (fn(&m->m2, dtype, 2, const_cast<void *>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    if (cols % GM_BK == 0) {
        const cuuint64_t dims[3] = {(cuuint64_t)GM_BK, (cuuint64_t)rows, (cuuint64_t)(cols / GM_BK)};
        const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, (cuuint64_t)GM_BK * 2};
        const cuuint32_t box[3] = {(cuuint32_t)GM_BK, (cuuint32_t)box_rows, 2};
        if (fn(&m->m3, dtype, 3, const_cast<void *>(base), dims, strides, box, es,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return false;
    }
    return true;
}

bool build_maps(sparsk_ctx *c)
{
    const sparsk_dims &d = c->dm;
    void *fp = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &qr) != cudaSuccess || !fp ||
        qr != cudaDriverEntryPointSuccess)
        return false;
    EncodeTiledFn fn = (EncodeTiledFn)fp;
    const int L = d.n_layers, V = d.vocab_text + d.vocab_speech;
    const size_t qd = (size_t)d.n_q_heads * d.head_dim, kd = (size_t)d.n_kv_heads * d.head_dim;
    bool ok = true;
    auto fill = [&](std::vector<TmaPair> &v, const std::vector<const bf16 *> &w, size_t rows, size_t cols, int box) {
        v.resize(L);
        for (int l = 0; l < L; l++) ok = ok && encode_maps(fn, &v[l], w[l], rows, cols, box);
    };
    fill(c->tm_wq, c->wq, qd, d.d_model, 2 * GM_BM); fill(c->tm_wk, c->wk, kd, d.d_model, 2 * GM_BM);
    fill(c->tm_wv, c->wv, kd, d.d_model, 2 * GM_BM); fill(c->tm_wo, c->wo, d.d_model, qd, 2 * GM_BM);
    fill(c->tm_wg, c->w_gate, d.d_ffn, d.d_model, GM_BM); fill(c->tm_wu, c->w_up, d.d_ffn, d.d_model, GM_BM);
    fill(c->tm_wd, c->w_down, d.d_model, d.d_ffn, 2 * GM_BM); fill(c->tm_head, c->head_proj, V, d.d_model, 2 * GM_BM);
    if (d.head_dim == 64 || d.head_dim == 128) {
        const size_t lstride = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len * d.head_dim;
        const size_t rows = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len;
        c->tm_kc16.resize(L);
        c->tm_vc16.resize(L);
        bool ok16 = rows < (1ull << 31);
        for (int l = 0; l < L && ok16; l++) {
            TmaPair t;
            ok16 = ok16 && encode_maps(fn, &t, c->kcache + l * lstride, rows, d.head_dim, AT_TP, CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
            c->tm_kc16[l] = d.head_dim == 128 ? t.m3 : t.m2;
            ok16 = ok16 && encode_maps(fn, &t, c->vcache + l * lstride, rows, d.head_dim, AT_TP, CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
            c->tm_vc16[l] = d.head_dim == 128 ? t.m3 : t.m2;
        }
        c->attn_tma_ok = ok16 ? 1 : 0;
    }
    if (d.head_dim == TA_HD) {
        const size_t lstride = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len * d.head_dim;
        c->tm_kc.resize(L);
        c->tm_vc.resize(L);
        for (int l = 0; l < L && ok; l++) {
            TmaPair t;
            ok = ok && encode_maps(fn, &t, c->kcache + l * lstride, (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len, d.head_dim, TA_NT,
                                   CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
            c->tm_kc[l] = t.m3;
            ok = ok && encode_maps(fn, &t, c->vcache + l * lstride, (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len, d.head_dim, TA_NT,
                                   CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
            c->tm_vc[l] = t.m3;
        }
    }
    for (int b = 0; b < 5; b++) {
        const int box = 16 << b;
        ok = ok && encode_maps(fn, &c->tm_x[b], c->xnorm, c->cap_rows, d.d_model, box);
        ok = ok && encode_maps(fn, &c->tm_ao[b], c->attn_o, c->cap_rows, qd, box);
        ok = ok && encode_maps(fn, &c->tm_act[b], c->act, c->cap_rows, d.d_ffn, box);
        ok = ok && encode_maps(fn, &c->tm_x_lo[b], c->xnorm_lo, c->cap_rows, d.d_model, box);
        ok = ok && encode_maps(fn, &c->tm_ao_lo[b], c->attn_o_lo, c->cap_rows, qd, box);
        ok = ok && encode_maps(fn, &c->tm_act_lo[b], c->act_lo, c->cap_rows, d.d_ffn, box);
    }
    return ok;
}

int box_index(int m_rows)
{
    int b = 0;
    while (b < 4 && (16 << b) < std::min(m_rows, GM_MAX_N)) b++;
    return b;
}

template <class Epi>
cudaError_t launch_gemm(sparsk_ctx *c, const TmaPair &a0, const TmaPair &a1, const TmaPair &a2, const TmaPair *b_maps,
                        const TmaPair *b_lo_maps, GemmArgs g, const Epi &epi)
{
    static PerDevice<bool> attr_done;
    bool &attr_set = attr_done.here();
    constexpr int SMEM_BUDGET = 220 * 1024;
    auto kern = wsgemm_kernel<Epi>;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BUDGET);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    const int bi = box_index(g.m_rows);
    g.box_n = 16 << bi;
    // the ring may be told to stay small enough for two CTAs (of this kernel or of the next one in
    // the stream) to share an SM, so that one's ending overlaps the other's first copies; rows
    // that do not fit such a ring take the whole SM
    auto stage_bytes = [&](int kb) { return 2 * kb * GM_BLK_BYTES + 2 * kb * g.box_n * GM_BK * 2; };
    auto plan = [&](int budget) {
        const int room = budget - 1024 - GM_XCHG_BYTES;
        // two k-blocks per copy whenever the inner dimension allows the 3-D view and two stages fit
        g.three_d = (g.K % GM_BK == 0) && 2 * stage_bytes(2) <= room && c->tc_kb != 1;
        g.kb = g.three_d ? 2 : 1;
        g.stages = std::min(GM_MAX_STAGES, room / stage_bytes(g.kb));
        return g.stages >= 2;
    };
    if (!plan(std::min(SMEM_BUDGET, c->gemm_smem_kb * 1024)) && !plan(SMEM_BUDGET)) return cudaErrorInvalidValue;
    g.status = c->sd.counts + CNT_STATUS;
    const int n_units = g.units[0] + (g.pair ? 0 : g.units[1] + g.units[2]);
    const int k_stages = ((g.K + GM_BK - 1) / GM_BK + g.kb - 1) / g.kb;
    g.splits = std::max(1, std::min(g.splits, k_stages));
    const size_t smem = 1024 + (size_t)g.stages * stage_bytes(g.kb) + GM_XCHG_BYTES;
    const int per_sm = (smem + 1024) * 2 <= 227 * 1024 ? std::max(1, c->gemm_cps) : 1;  // CTAs of this launch that fit an SM
    const int grid_x = std::max(1, std::min(c->n_sm * per_sm, n_units * g.splits));
    const int grid_y = (g.m_rows + GM_MAX_N - 1) / GM_MAX_N;
    if (g.three_d)
        return launch(c, kern, dim3(grid_x, grid_y), dim3(GM_THREADS), smem, a0.m3, a1.m3, a2.m3, b_maps[bi].m3,
                      b_lo_maps[bi].m3, g, epi);
    return launch(c, kern, dim3(grid_x, grid_y), dim3(GM_THREADS), smem, a0.m2, a1.m2, a2.m2, b_maps[bi].m2,
                  b_lo_maps[bi].m2, g, epi);
}

int div_up(int a, int b) { return (a + b - 1) / b; }

cudaError_t run_norm(sparsk_ctx *c, const float *h, const bf16 *gain, const int *row_idx, int n_rows)
{
    return launch(c, rmsnorm_rows_kernel, dim3(n_rows), dim3(256), 0, h, gain, row_idx, c->xnorm, c->xnorm_lo, n_rows,
                  c->dm.d_model, c->dm.rms_eps);
}

// How many cuts of the inner dimension fill the machine when a product has `units` units.
int splits_for(const sparsk_ctx *c, int units)
{
    const int ctas = c->n_sm * std::max(1, c->gemm_cps);
    return units * 2 <= ctas ? ctas / units : 1;
}

// One transformer layer over a row set on the tensor-core path, in two halves: the front
// (RMSNorm, q/k/v projection, rotary embedding, cache append) and the back (attention,
// O-projection, MLP).  The last layer of an upper pass runs its back half on fewer rows.
cudaError_t run_layer_tc_front(sparsk_ctx *c, int layer, float *h, const RowSet &rs)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1, M = rs.n_rows;
    const int qd = d.n_q_heads * d.head_dim, kd = d.n_kv_heads * d.head_dim;
    const size_t lstride = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len * d.head_dim;
    kv_t *kc = c->kcache + li * lstride, *vc = c->vcache + li * lstride;
    cudaError_t e;
    c->cur_class = KC_MISC;
    if ((e = run_norm(c, h, c->attn_norm[li], nullptr, M)) != cudaSuccess) return e;
    {
        c->cur_class = KC_QKV;
        GemmArgs g{};
        g.K = d.d_model; g.units[0] = div_up(qd, 2 * GM_BM); g.units[1] = g.units[2] = div_up(kd, 2 * GM_BM);
        g.m_rows = M;
        g.splits = splits_for(c, g.units[0] + g.units[1] + g.units[2]);
        QkvEnd ep;
        ep.q_out = c->qbuf; ep.kc = kc; ep.vc = vc; ep.rope = c->rope;
        ep.row_slot = rs.slot; ep.row_pos = rs.pos; ep.Hq = d.n_q_heads; ep.Hkv = d.n_kv_heads; ep.hd = d.head_dim;
        ep.S = d.max_seq_len; ep.partial = g.splits > 1 ? c->qkv_part : nullptr;
        if ((e = launch_gemm(c, c->tm_wq[li], c->tm_wk[li], c->tm_wv[li], c->tm_x, c->tm_x_lo, g, ep)) != cudaSuccess) return e;
        if (g.splits > 1 &&
            (e = launch(c, qkv_finish_kernel, dim3(M), dim3(256), 0, c->qkv_part, c->qbuf, kc, vc, (const float2 *)c->rope,
                        rs.slot, rs.pos, M, d.n_q_heads, d.n_kv_heads, d.head_dim, d.max_seq_len)) != cudaSuccess)
            return e;
    }
    c->cur_class = KC_MISC;
    return cudaSuccess;
}

cudaError_t run_layer_tc_back(sparsk_ctx *c, int layer, float *h, const RowSet &rs)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1, M = rs.n_rows;
    const int qd = d.n_q_heads * d.head_dim;
    cudaError_t e;
    c->cur_class = KC_ATTN;
    if ((e = run_attn(c, layer, rs)) != cudaSuccess) return e;
    {
        c->cur_class = KC_OPROJ;
        GemmArgs g{};
        g.K = qd; g.units[0] = div_up(d.d_model, 2 * GM_BM); g.m_rows = M;
        g.splits = splits_for(c, g.units[0]);
        ResidEnd ep;
        ep.h = h; ep.n_out = d.d_model; ep.atomic = 1;
        if ((e = launch_gemm(c, c->tm_wo[li], c->tm_wo[li], c->tm_wo[li], c->tm_ao, c->tm_ao_lo, g, ep)) != cudaSuccess) return e;
    }
    c->cur_class = KC_MISC;
    if ((e = run_norm(c, h, c->mlp_norm[li], nullptr, M)) != cudaSuccess) return e;
    {
        c->cur_class = KC_GATEUP;
        GemmArgs g{};
        g.K = d.d_model; g.units[0] = div_up(d.d_ffn, GM_BM); g.pair = 1; g.m_rows = M; g.splits = 1;
        GateUpEnd ep;
        ep.u = c->act; ep.u_lo = c->act_lo; ep.F = d.d_ffn;
        if ((e = launch_gemm(c, c->tm_wg[li], c->tm_wu[li], c->tm_wu[li], c->tm_x, c->tm_x_lo, g, ep)) != cudaSuccess) return e;
    }
    {
        c->cur_class = KC_DOWN;
        GemmArgs g{};
        g.K = d.d_ffn; g.units[0] = div_up(d.d_model, 2 * GM_BM); g.m_rows = M;
        g.splits = splits_for(c, g.units[0]);
        ResidEnd ep;
        ep.h = h; ep.n_out = d.d_model; ep.atomic = 1;
        e = launch_gemm(c, c->tm_wd[li], c->tm_wd[li], c->tm_wd[li], c->tm_act, c->tm_act_lo, g, ep);
    }
    c->cur_class = KC_MISC;
    return e;
}

bool use_tc(const sparsk_ctx *c, int n_rows) { return c->tc_ok && n_rows >= c->gemm_min_rows && c->dm.d_model >= GM_BK; }


// Head of `layer` over list `l` on the tensor-core path.
cudaError_t run_head_tc(sparsk_ctx *c, int layer, const float *h, int list, int n_rows)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1, B = d.max_seqs, speech = list & 1;
    cudaError_t e;
    c->cur_class = KC_MISC;
    if ((e = run_norm(c, h, c->head_norm[li], c->sd.list_row + (size_t)list * B, n_rows)) != cudaSuccess) return e;
    c->cur_class = KC_HEAD;
    HeadEnd ep;
    ep.seq_of_row = c->sd.list_seq + (size_t)list * B; ep.argmax = c->sd.argmax; ep.logits = head_logits(c);
    ep.lo = speech ? d.vocab_text : 0; ep.hi = speech ? d.vocab_text + d.vocab_speech : d.vocab_text;
    ep.V = d.vocab_text + d.vocab_speech;
    GemmArgs g{};
    g.K = d.d_model; g.units[0] = div_up(ep.hi - ep.lo, 2 * GM_BM); g.row0[0] = ep.lo; g.m_rows = n_rows;
    g.splits = 1;
    e = launch_gemm(c, c->tm_head[li], c->tm_head[li], c->tm_head[li], c->tm_x, c->tm_x_lo, g, ep);
    c->cur_class = KC_MISC;
    return e;
}


// ---------------------------------------------------------------- persistent layer-range kernel
bool build_mega(sparsk_ctx *c)
{
    const sparsk_dims &d = c->dm;
    void *fp = nullptr;
    cudaDriverEntryPointQueryResult qr;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &qr) != cudaSuccess || !fp ||
        qr != cudaDriverEntryPointSuccess)
        return false;
    EncodeTiledFn fn = (EncodeTiledFn)fp;
    const size_t qd = (size_t)d.n_q_heads * d.head_dim, kd = (size_t)d.n_kv_heads * d.head_dim;
    const size_t lstride = (size_t)d.max_seqs * d.n_kv_heads * d.max_seq_len * d.head_dim;
    // [16 rows][256 columns] boxes of a row-major matrix, no swizzle, zero fill outside
    auto enc = [&](CUtensorMap *m, const void *base, size_t rows, size_t cols) {
        const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
        const cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
        const cuuint32_t box[2] = {(cuuint32_t)MK_BOX_COLS, (cuuint32_t)MK_BOX_ROWS};
        const cuuint32_t es[2] = {1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    // the swizzled three-dimensional view needs inner dimensions that are whole 64-element blocks
    c->mk_tc_ok = d.d_model % 64 == 0 && d.d_ffn % 64 == 0 && qd % 64 == 0;
    auto enc_sw = [&](CUtensorMap *m, const void *base, size_t rows, size_t cols) {
        const cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
        const cuuint64_t strides[2] = {(cuuint64_t)cols * 2, 128};
        const cuuint32_t box[3] = {64, (cuuint32_t)MK_BOX_ROWS, (cuuint32_t)(MK_BOX_COLS / 64)};
        const cuuint32_t es[3] = {1, 1, 1};
        return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(base), dims, strides, box, es,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
    };
    c->mk_host.resize(d.n_layers);
    bool ok = true;
    for (int l = 0; l < d.n_layers; l++) {
        MkLayer &m = c->mk_host[l];
        memset(&m, 0, sizeof m);
        const void *mats[MKW_N] = {c->wq[l], c->wk[l], c->wv[l], c->wo[l], c->w_gate[l], c->w_up[l], c->w_down[l]};
        const size_t rows[MKW_N] = {qd, kd, kd, (size_t)d.d_model, (size_t)d.d_ffn, (size_t)d.d_ffn, (size_t)d.d_model};
        const size_t cols[MKW_N] = {(size_t)d.d_model, (size_t)d.d_model, (size_t)d.d_model, qd, (size_t)d.d_model,
                                    (size_t)d.d_model, (size_t)d.d_ffn};
        for (int k = 0; k < MKW_N; k++) {
            ok = ok && enc(&m.map[k], mats[k], rows[k], cols[k]);
            if (c->mk_tc_ok) ok = ok && enc_sw(&m.map[MKW_N + k], mats[k], rows[k], cols[k]);
        }
        m.attn_gain = c->attn_norm[l];
        m.mlp_gain = c->mlp_norm[l];
        m.kc = c->kcache + l * lstride;
        m.vc = c->vcache + l * lstride;
    }
    if (!ok) return false;
    if (cudaMemcpyAsync(c->mk_layers, c->mk_host.data(), sizeof(MkLayer) * d.n_layers, cudaMemcpyHostToDevice,
                        c->stream) != cudaSuccess ||
        cudaMemsetAsync(c->mk_bar, 0, sizeof(unsigned long long), c->stream) != cudaSuccess ||
        cudaMemsetAsync(c->mk_abort, 0, sizeof(int), c->stream) != cudaSuccess)
        return false;
    c->mk_bar_base = 0;
    int dev = 0, coop = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess)
        return false;
    c->mk_coop = coop;
    return true;
}

size_t mega_smem(const sparsk_dims &) { return (size_t)MK_SLOTS * MK_SLOT_BYTES + MK_AREA_BYTES + 1024; }

// Can a pass of n_rows rows go through the persistent kernel?
bool use_mega(const sparsk_ctx *c, int n_rows)
{
    return c->mega && c->mk_ok && c->mk_coop && n_rows >= 1 && n_rows <= c->mk_max_rows && (n_rows <= 2 || c->mk_tc_ok) &&
           mk_attn_bytes(c->dm.head_dim) <= MK_AREA_BYTES && c->dm.head_dim % (2 * MK_BOX_ROWS) == 0;
}

template <int M, int HD>
cudaError_t launch_mega_inst(sparsk_ctx *c, const MkArgs &a, size_t smem)
{
    static PerDevice<int> grid_dev;  // 0: not asked yet, 1: one CTA per SM fits, 2: it does not
    int &grid_ok = grid_dev.here();
    auto kern = mega_kernel<M, HD>;
    if (grid_ok == 0) {
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        int per_sm = 0;
        e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, MK_THREADS, smem);
        if (e != cudaSuccess) return e;
        grid_ok = per_sm >= 1 ? 1 : 2;
    }
    if (grid_ok != 1) return cudaErrorCooperativeLaunchTooLarge;
    cudaLaunchConfig_t cfg;
    memset(&cfg, 0, sizeof cfg);
    cfg.gridDim = dim3(c->n_sm);
    cfg.blockDim = dim3(MK_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = c->stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    c->launches++;
    const bool timed = (c->time_class == KC_MEGA || c->time_class == KC_ALL) && c->tev_used + 2 <= c->tev.size();
    if (timed) {
        c->tev_class[c->tev_used / 2] = KC_MEGA;
        cudaEventRecord(c->tev[c->tev_used++], c->stream);
    }
    const cudaError_t e = cudaLaunchKernelEx(&cfg, kern, a);
    if (timed) cudaEventRecord(c->tev[c->tev_used++], c->stream);
    return e;
}

// Layers [l_begin, l_end) (0-based) over a row set of one or two rows, in one launch.
cudaError_t run_mega(sparsk_ctx *c, int l_begin, int l_end, float *h, const RowSet &rs)
{
    const sparsk_dims &d = c->dm;
    MkArgs a{};
    a.layers = c->mk_layers; a.layer_begin = l_begin; a.layer_end = l_end; a.h = h;
    a.row_slot = rs.slot; a.row_pos = rs.pos; a.grp_row0 = rs.grp_row0; a.grp_nrows = rs.grp_nrows;
    a.n_rows = rs.n_rows; a.n_groups = rs.n_groups_h;
    a.q_buf = c->qbuf; a.attn_o = c->mk_attn_o; a.act = c->mk_act; a.part_o = c->part_o; a.part_ml = c->part_ml;
    a.rope = c->rope;
    a.d = d.d_model; a.Hq = d.n_q_heads; a.Hkv = d.n_kv_heads; a.hd = d.head_dim; a.F = d.d_ffn; a.S = d.max_seq_len;
    a.n_slots = d.max_seqs; a.eps = d.rms_eps;
    // KV cut: an item for every attention warp of the machine if there are that many 16-position tiles
    const int G = d.n_q_heads / d.n_kv_heads;
    const int n_qblk = (rs.max_grp_rows * G + 15) / 16;
    const int base = std::max(1, rs.n_groups_h * n_qblk * d.n_kv_heads);
    const int tiles = std::max(1, (rs.max_len + AT_TP - 1) / AT_TP);
    int splits = c->attn_split > 0 ? (rs.max_len + c->attn_split - 1) / c->attn_split
                                   : (c->n_sm * MK_ATT_WARPS + base - 1) / base;
    splits = std::max(1, std::min(splits, std::min(MK_MAX_SPLITS, tiles)));
    a.att_qblk = n_qblk;
    a.att_split_len = ((rs.max_len + splits - 1) / splits + AT_TP - 1) / AT_TP * AT_TP;
    a.att_splits = std::max(1, (rs.max_len + a.att_split_len - 1) / a.att_split_len);
    a.bar = c->mk_bar; a.bar_base = c->mk_bar_base; a.abort_word = c->mk_abort; a.status = c->sd.counts + CNT_STATUS;
    if (c->inject_timeout) {
        // the launch is told a barrier count that is never reached: its first grid barrier runs
        // into the wall-clock limit, every CTA gives up and the step reports SPARSK_ETIMEOUT
        a.bar_base += 1ull << 40;
        c->inject_timeout = 0;
    }
    a.trace = c->mk_trace;
    c->mk_trace_n = 1 + 6 * (l_end - l_begin);
    c->mk_bar_base += 6ull * (unsigned long long)(l_end - l_begin) * (unsigned long long)c->n_sm;
    const size_t smem = mega_smem(d);
    if (d.head_dim == 128) {
        switch (rs.n_rows) {
        case 1: return launch_mega_inst<1, 128>(c, a, smem);
        case 2: return launch_mega_inst<2, 128>(c, a, smem);
        case 3: return launch_mega_inst<3, 128>(c, a, smem);
        default: return launch_mega_inst<4, 128>(c, a, smem);
        }
    }
    switch (rs.n_rows) {
    case 1: return launch_mega_inst<1, 64>(c, a, smem);
    case 2: return launch_mega_inst<2, 64>(c, a, smem);
    case 3: return launch_mega_inst<3, 64>(c, a, smem);
    default: return launch_mega_inst<4, 64>(c, a, smem);
    }
}

// Front half of a layer over a row set: q to the query buffer, k and v into the cache.
cudaError_t run_layer_front(sparsk_ctx *c, int layer, float *h, const RowSet &rs)
{
    if (use_tc(c, rs.n_rows)) return run_layer_tc_front(c, layer, h, rs);
    c->cur_class = KC_QKV;
    const cudaError_t e = run_qkv(c, layer, h, rs);
    c->cur_class = KC_MISC;
    return e;
}

// Back half: attention, O-projection and MLP; h <- h^(layer).
cudaError_t run_layer_back(sparsk_ctx *c, int layer, float *h, const RowSet &rs)
{
    const sparsk_dims &d = c->dm;
    const int li = layer - 1;
    cudaError_t e;
    if (use_tc(c, rs.n_rows)) return run_layer_tc_back(c, layer, h, rs);
    c->cur_class = KC_ATTN;
    if ((e = run_attn(c, layer, rs)) != cudaSuccess) return e;
    c->cur_class = KC_OPROJ;
    if ((e = run_resid(c, c->wo[li], c->attn_o, h, d.n_q_heads * d.head_dim, d.d_model, rs.n_rows)) != cudaSuccess) return e;
    c->cur_class = KC_GATEUP;
    if ((e = run_gateup(c, layer, h, rs.n_rows)) != cudaSuccess) return e;
    c->cur_class = KC_DOWN;
    e = run_resid(c, c->w_down[li], c->act, h, d.d_ffn, d.d_model, rs.n_rows);
    c->cur_class = KC_MISC;
    return e;
}

// One transformer layer over a row set: h <- h^(layer).
cudaError_t run_layer(sparsk_ctx *c, int layer, float *h, const RowSet &rs)
{
    const cudaError_t e = run_layer_front(c, layer, h, rs);
    return e != cudaSuccess ? e : run_layer_back(c, layer, h, rs);
}

// Layers l_first..l_last (1-based, inclusive) over a row set.
cudaError_t run_layers(sparsk_ctx *c, int l_first, int l_last, float *h, const RowSet &rs)
{
    if (l_first > l_last) return cudaSuccess;
    const int n_layers = l_last - l_first + 1;
    if (use_mega(c, rs.n_rows)) {
        c->route_layers[0] += n_layers;
        return run_mega(c, l_first - 1, l_last, h, rs);
    }
    c->route_layers[use_tc(c, rs.n_rows) ? 1 : 2] += n_layers;
    for (int l = l_first; l <= l_last; l++) {
        const cudaError_t e = run_layer(c, l, h, rs);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

bool good(const sparsk_ctx *c) { return c && c->magic == CTX_MAGIC; }

}  // namespace

// =============================================================================== C ABI

extern "C" size_t sparsk_workspace_bytes(const sparsk_dims *dims)
{
    if (!dims_ok(dims)) return 0;
    return carve(nullptr, dims, nullptr);
}

extern "C" int sparsk_create(const sparsk_dims *dims, const sparsk_weights *w, void *workspace,
                             size_t workspace_bytes, void *cuda_stream, sparsk_ctx **out)
{
    if (!out) return SPARSK_EINVAL;
    *out = nullptr;
    if (!dims_ok(dims) || !w || !workspace) return SPARSK_EINVAL;
    if ((uintptr_t)workspace % 256) return SPARSK_EINVAL;
    if (workspace_bytes < sparsk_workspace_bytes(dims)) return SPARSK_EINVAL;
    const int L = dims->n_layers, e = dims->exit_layer;
    const void *const *arrs[] = {w->attn_norm, w->wq, w->wk, w->wv, w->wo, w->mlp_norm, w->w_gate, w->w_up, w->w_down};
    if (!w->embed || ((uintptr_t)w->embed % 16) || !w->head_norm || !w->head_proj) return SPARSK_EINVAL;
    for (auto a : arrs) {
        if (!a) return SPARSK_EINVAL;
        for (int l = 0; l < L; l++)
            if (!a[l] || ((uintptr_t)a[l] % 16)) return SPARSK_EINVAL;
    }
    for (int l = 0; l < L; l++)
        if (((uintptr_t)w->head_norm[l] % 16) || ((uintptr_t)w->head_proj[l] % 16)) return SPARSK_EINVAL;
    if (((size_t)dims->vocab_text * dims->d_model * 2) % 16) return SPARSK_EINVAL;
    // the heads of layers e and L are what the periodic schedule reads
    if (!w->head_norm[L - 1] || !w->head_proj[L - 1]) return SPARSK_ENOHEAD;
    if (dims->refresh_period > 1 && e < L && (!w->head_norm[e - 1] || !w->head_proj[e - 1])) return SPARSK_ENOHEAD;
    if (dims->conf_modalities)   // the confidence rule consults the head of every layer from conf_start on
        for (int l = dims->conf_start; l < L; l++)
            if (!w->head_norm[l - 1] || !w->head_proj[l - 1]) return SPARSK_ENOHEAD;

    sparsk_ctx *ctx = new (std::nothrow) sparsk_ctx();
    if (!ctx) return SPARSK_EINVAL;
    ctx->magic = CTX_MAGIC;
    ctx->dm = *dims;
    if (ctx->dm.prefill_rows <= 0) ctx->dm.prefill_rows = 64;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->err[0] = 0;
    auto cp = [&](std::vector<const bf16 *> &dst, const void *const *src) {
        dst.resize(L);
        for (int l = 0; l < L; l++) dst[l] = (const bf16 *)src[l];
    };
    cp(ctx->attn_norm, w->attn_norm); cp(ctx->wq, w->wq); cp(ctx->wk, w->wk); cp(ctx->wv, w->wv);
    cp(ctx->wo, w->wo); cp(ctx->mlp_norm, w->mlp_norm); cp(ctx->w_gate, w->w_gate); cp(ctx->w_up, w->w_up);
    cp(ctx->w_down, w->w_down); cp(ctx->head_norm, w->head_norm); cp(ctx->head_proj, w->head_proj);
    ctx->embed = (const bf16 *)w->embed;
    ctx->cap_rows = cap_rows_of(&ctx->dm);
    carve(ctx, &ctx->dm, (char *)workspace);
    ctx->h_len.assign(dims->max_seqs, 0);
    ctx->h_pend.assign(dims->max_seqs, 0);
    ctx->pdl = 1; ctx->attn_split = 0; ctx->gemm_min_rows = 3;
    ctx->tc_ok = false;
    ctx->tc_kb = 0;
    ctx->gemm_smem_kb = 220;
    ctx->gemm_cps = 1;
    ctx->mk_max_rows = MK_MAX_ROWS;
    ctx->attn_tc = 1; ctx->attn_tc_min_q = 33; ctx->attn_stages = AW_NST;
    ctx->inject_timeout = 0;
    ctx->attn_ticket_base = 0; ctx->attn_dynamic = 1; ctx->attn_ctas = 0;
    ctx->attn_tma = 1; ctx->attn_tma_ok = 0;
    ctx->trim_last = 1;
    ctx->conf_host = nullptr; ctx->conf_ent_host = nullptr;
    ctx->h_fill.assign(dims->max_seqs, std::vector<int>());
    for (auto &v : ctx->route_layers) v = 0;
    ctx->mega = 1; ctx->mk_ok = 0; ctx->mk_coop = 0; ctx->mk_bar_base = 0; ctx->mk_trace_n = 0;
    ctx->gv_ks = 0; ctx->gv_r = 0;
    ctx->dbg_hidden = nullptr; ctx->dbg_logits = nullptr;
    ctx->samp_temperature = 0.f; ctx->samp_top_p = 1.f; ctx->samp_uniforms = nullptr; ctx->samp_scratch = nullptr;
    ctx->launches = 0;
    ctx->cur_class = KC_MISC; ctx->time_class = KC_MISC; ctx->tev_used = 0;
    ctx->stage_next = 0;
    for (int i = 0; i < STAGE_RING; i++) { ctx->stage_host[i] = nullptr; ctx->stage_ev[i] = nullptr; }
    ctx->io_host = nullptr;

    int rc = SPARSK_OK;
    do {
        int dev = 0;
        cudaError_t ce;
        if ((ce = cudaGetDevice(&dev)) != cudaSuccess ||
            (ce = cudaDeviceGetAttribute(&ctx->n_sm, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) {
            rc = fail(ctx, SPARSK_ECUDA, "device query failed: %s", cudaGetErrorString(ce));
            break;
        }
        for (int i = 0; i < STAGE_RING && rc == SPARSK_OK; i++) {
            if ((ce = cudaHostAlloc((void **)&ctx->stage_host[i], 3 * sizeof(int) * dims->max_seqs, cudaHostAllocDefault)) != cudaSuccess ||
                (ce = cudaEventCreateWithFlags(&ctx->stage_ev[i], cudaEventDisableTiming)) != cudaSuccess)
                rc = fail(ctx, SPARSK_ECUDA, "staging setup failed: %s", cudaGetErrorString(ce));
        }
        if (rc == SPARSK_OK &&
            (ce = cudaHostAlloc((void **)&ctx->io_host, sizeof(int) * (3 * (size_t)dims->max_seqs + 1), cudaHostAllocDefault)) != cudaSuccess)
            rc = fail(ctx, SPARSK_ECUDA, "staging setup failed: %s", cudaGetErrorString(ce));
        if (rc) break;
        if (dims->conf_modalities) {
            // one region per segment of a step (at most one per layer, plus lists per consulted layer)
            ctx->conf_seg_ints = 4 * (size_t)ctx->cap_rows + 4 * (size_t)dims->max_seqs + 8;
            ctx->conf_host_ints = ctx->conf_seg_ints * (2 * (size_t)L + 4);
            if ((ce = cudaHostAlloc((void **)&ctx->conf_host, ctx->conf_host_ints * sizeof(int), cudaHostAllocDefault)) != cudaSuccess ||
                (ce = cudaHostAlloc((void **)&ctx->conf_ent_host, sizeof(float) * dims->max_seqs, cudaHostAllocDefault)) != cudaSuccess) {
                rc = fail(ctx, SPARSK_ECUDA, "staging setup failed: %s", cudaGetErrorString(ce));
                break;
            }
        }
        // no silent change of path: without TMA descriptors the batched path cannot run
        ctx->tc_ok = build_maps(ctx);
        if (!ctx->tc_ok) {
            rc = fail(ctx, SPARSK_ECUDA, "building the TMA descriptors failed");
            break;
        }
        ctx->mk_ok = build_mega(ctx) ? 1 : 0;
        if (!ctx->mk_ok) {
            rc = fail(ctx, SPARSK_ECUDA, "setting up the persistent layer kernel failed");
            break;
        }
        // rotary table in double, stored as float (cos, sin)
        const int half = dims->head_dim / 2;
        std::vector<float2> tab((size_t)dims->max_seq_len * half);
        for (int i = 0; i < half; i++) {
            const double inv = std::pow((double)dims->rope_base, -2.0 * i / dims->head_dim);
            for (int p = 0; p < dims->max_seq_len; p++) {
                const double th = (double)p * inv;
                tab[(size_t)p * half + i] = make_float2((float)std::cos(th), (float)std::sin(th));
            }
        }
        if ((ce = cudaMemcpyAsync(ctx->rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice, ctx->stream)) != cudaSuccess ||
            // the cache starts out as zeros: the tcgen05 attention kernel multiplies whole 64-position
            // tiles, and a masked weight of zero times an unwritten NaN pattern would still be NaN
            (ce = cudaMemsetAsync(ctx->kcache, 0, sizeof(kv_t) * (size_t)dims->n_layers * dims->max_seqs * dims->n_kv_heads * dims->max_seq_len * dims->head_dim, ctx->stream)) != cudaSuccess ||
            (ce = cudaMemsetAsync(ctx->vcache, 0, sizeof(kv_t) * (size_t)dims->n_layers * dims->max_seqs * dims->n_kv_heads * dims->max_seq_len * dims->head_dim, ctx->stream)) != cudaSuccess ||
            (ce = cudaMemsetAsync(ctx->kv_len, 0, sizeof(int) * dims->max_seqs, ctx->stream)) != cudaSuccess ||
            (ce = cudaMemsetAsync(ctx->pend_cnt, 0, sizeof(int) * dims->max_seqs, ctx->stream)) != cudaSuccess ||
            (ce = cudaMemsetAsync(ctx->sd.counts, 0, sizeof(int) * 8, ctx->stream)) != cudaSuccess ||
            (ce = cudaMemsetAsync(ctx->attn_ticket, 0, sizeof(unsigned), ctx->stream)) != cudaSuccess ||
            (ce = cudaMemsetAsync(ctx->qkv_part, 0, sizeof(float) * (size_t)ctx->cap_rows * (dims->n_q_heads + 2 * dims->n_kv_heads) * dims->head_dim, ctx->stream)) != cudaSuccess ||
            (ce = cudaStreamSynchronize(ctx->stream)) != cudaSuccess) {
            rc = fail(ctx, SPARSK_ECUDA, "table upload failed: %s", cudaGetErrorString(ce));
            break;
        }
    } while (0);
    if (rc != SPARSK_OK) {
        sparsk_destroy(ctx);
        return rc;
    }
    *out = ctx;
    return SPARSK_OK;
}

extern "C" int sparsk_destroy(sparsk_ctx *ctx)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    cudaStreamSynchronize(ctx->stream);
    for (int i = 0; i < STAGE_RING; i++) {
        if (ctx->stage_host[i]) cudaFreeHost(ctx->stage_host[i]);
        if (ctx->stage_ev[i]) cudaEventDestroy(ctx->stage_ev[i]);
    }
    if (ctx->io_host) cudaFreeHost(ctx->io_host);
    for (cudaEvent_t ev : ctx->tev) cudaEventDestroy(ev);
    if (ctx->conf_host) cudaFreeHost(ctx->conf_host);
    if (ctx->conf_ent_host) cudaFreeHost(ctx->conf_ent_host);
    ctx->magic = 0;
    delete ctx;
    return SPARSK_OK;
}

extern "C" const char *sparsk_last_error(const sparsk_ctx *ctx) { return good(ctx) ? ctx->err : "invalid context"; }
extern "C" int64_t sparsk_launch_count(const sparsk_ctx *ctx) { return good(ctx) ? ctx->launches : -1; }
extern "C" int sparsk_conf_entropies(const sparsk_ctx *ctx, int32_t n_seqs, float *out)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    const int L = ctx->dm.n_layers;
    if (!out || n_seqs < 0 || (size_t)n_seqs * L > ctx->conf_trace.size()) return SPARSK_EINVAL;
    for (size_t k = 0; k < (size_t)n_seqs * L; k++) out[k] = ctx->conf_trace[k];
    return SPARSK_OK;
}
extern "C" int sparsk_route_counts(const sparsk_ctx *ctx, int64_t *layer_passes)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (!layer_passes) return SPARSK_EINVAL;
    for (int i = 0; i < 3; i++) layer_passes[i] = ctx->route_layers[i];
    return SPARSK_OK;
}

extern "C" int sparsk_set_debug(sparsk_ctx *ctx, float *exit_hidden, float *exit_logits)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    ctx->dbg_hidden = exit_hidden;
    ctx->dbg_logits = exit_logits;
    return SPARSK_OK;
}

extern "C" size_t sparsk_sampling_scratch_bytes(const sparsk_dims *dims)
{
    if (!dims_ok(dims)) return 0;
    return (size_t)dims->max_seqs * ((size_t)dims->vocab_text + dims->vocab_speech) * sizeof(float);
}

extern "C" int sparsk_set_sampling(sparsk_ctx *ctx, float temperature, float top_p, const float *uniforms, void *scratch,
                                   size_t scratch_bytes)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (!uniforms) {  // back to greedy decoding
        ctx->samp_uniforms = nullptr;
        ctx->samp_scratch = nullptr;
        return SPARSK_OK;
    }
    if (ctx->dm.conf_modalities)
        return fail(ctx, SPARSK_EINVAL, "set_sampling: a context with confidence-based exit decodes greedily");
    if (!(temperature > 0.f) || !(temperature < INFINITY) || !(top_p > 0.f) || !(top_p <= 1.f))
        return fail(ctx, SPARSK_EINVAL, "set_sampling: temperature %g, top_p %g", (double)temperature, (double)top_p);
    if (ctx->dm.vocab_text > SP_MAX_RANGE || ctx->dm.vocab_speech > SP_MAX_RANGE)
        return fail(ctx, SPARSK_ECAPACITY, "set_sampling: a modality has more than %d ids", SP_MAX_RANGE);
    if (!scratch || ((uintptr_t)scratch % 16) || scratch_bytes < sparsk_sampling_scratch_bytes(&ctx->dm))
        return fail(ctx, SPARSK_EINVAL, "set_sampling: scratch of %zu bytes, need %zu (16-byte aligned)", scratch_bytes,
                    sparsk_sampling_scratch_bytes(&ctx->dm));
    ctx->samp_temperature = temperature;
    ctx->samp_top_p = top_p;
    ctx->samp_uniforms = uniforms;
    ctx->samp_scratch = (float *)scratch;
    return SPARSK_OK;
}

extern "C" int sparsk_set_option(sparsk_ctx *ctx, const char *name, int64_t value)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (!name) return fail(ctx, SPARSK_EINVAL, "option name is NULL");
    if (!strcmp(name, "gemm_min_rows") && value >= 1) ctx->gemm_min_rows = (int)std::min<int64_t>(value, 1 << 30);
    else if (!strcmp(name, "pdl") && (value == 0 || value == 1)) ctx->pdl = (int)value;
    else if (!strcmp(name, "attn_split") && value >= 0 && value <= (1 << 24)) ctx->attn_split = (int)value;
    else if (!strcmp(name, "gemv_ks") && (value == 0 || value == 1 || value == 2 || value == 4 || value == 8 || value == 16)) ctx->gv_ks = (int)value;
    else if (!strcmp(name, "mega") && (value == 0 || value == 1)) ctx->mega = (int)value;
    else if (!strcmp(name, "attn_stages") && (value == 2 || value == 3)) ctx->attn_stages = (int)value;
    else if (!strcmp(name, "attn_dynamic") && (value == 0 || value == 1)) ctx->attn_dynamic = (int)value;
    else if (!strcmp(name, "attn_tma") && (value == 0 || value == 1)) ctx->attn_tma = (int)value;
    else if (!strcmp(name, "attn_ctas") && value >= 0 && value <= 65535) ctx->attn_ctas = (int)value;
    else if (!strcmp(name, "attn_tc") && (value == 0 || value == 1)) ctx->attn_tc = (int)value;
    else if (!strcmp(name, "attn_tc_min_q") && value >= 1 && value <= (1 << 20)) ctx->attn_tc_min_q = (int)value;
    else if (!strcmp(name, "mega_max_rows") && value >= 1 && value <= MK_MAX_ROWS) ctx->mk_max_rows = (int)value;
    else if (!strcmp(name, "gemm_kb") && (value == 0 || value == 1)) ctx->tc_kb = (int)value;
    else if (!strcmp(name, "gemm_ctas_per_sm") && (value == 1 || value == 2)) ctx->gemm_cps = (int)value;
    else if (!strcmp(name, "gemm_smem_kb") && value >= 48 && value <= 220) ctx->gemm_smem_kb = (int)value;
    else if (!strcmp(name, "trim_last_layer") && value >= 0 && value <= 2) ctx->trim_last = (int)value;
    else if (!strcmp(name, "inject_barrier_timeout") && (value == 0 || value == 1)) ctx->inject_timeout = (int)value;
    else if (!strcmp(name, "gemv_r") && (value == 0 || value == 1 || value == 2 || value == 4)) ctx->gv_r = (int)value;
    else if (!strcmp(name, "time_kernel") && value >= 0 && value <= KC_ALL) {
        // start (or stop, with 0) timing every launch of one kernel class; resets the totals
        if (value && ctx->tev.empty()) {
            ctx->tev.resize(2 * TIME_POOL);
            ctx->tev_class.assign(TIME_POOL, 0);
            for (auto &ev : ctx->tev) CU(cudaEventCreate(&ev));
        }
        ctx->time_class = (int)value;
        ctx->tev_used = 0;
    } else return fail(ctx, SPARSK_EINVAL, "unknown option or bad value: %s=%lld", name, (long long)value);
    return SPARSK_OK;
}

extern "C" int sparsk_kernel_time(sparsk_ctx *ctx, double *total_ms, int64_t *n_launches)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (!total_ms || !n_launches) return fail(ctx, SPARSK_EINVAL, "kernel_time: NULL output");
    CU(cudaStreamSynchronize(ctx->stream));
    double tot = 0.0;
    for (size_t i = 0; i + 1 < ctx->tev_used; i += 2) {
        float ms = 0.f;
        CU(cudaEventElapsedTime(&ms, ctx->tev[i], ctx->tev[i + 1]));
        tot += ms;
    }
    *total_ms = tot;
    *n_launches = (int64_t)(ctx->tev_used / 2);
    return SPARSK_OK;
}

// Reads and clears the device status word (the stream is synchronised) and turns it into a
// return code.  After a timeout the persistent kernels' grid-barrier counter, its host mirror and
// the abort word start over, so that the next launch does not find a stale abort request or a
// counter that no longer matches its base.
static int act_on_status(sparsk_ctx *ctx, int status);
static int read_status(sparsk_ctx *ctx)
{
    int status = 0;
    CU(cudaMemcpyAsync(&status, ctx->sd.counts + CNT_STATUS, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    return act_on_status(ctx, status);
}
// What a status word read back from the device (the stream is idle) means for the caller.
static int act_on_status(sparsk_ctx *ctx, int status)
{
    if (status) CU(cudaMemsetAsync(ctx->sd.counts + CNT_STATUS, 0, sizeof(int), ctx->stream));
    if (status & ST_TIMEOUT) {
        CU(cudaMemsetAsync(ctx->mk_bar, 0, sizeof(unsigned long long), ctx->stream));
        CU(cudaMemsetAsync(ctx->mk_abort, 0, sizeof(int), ctx->stream));
        CU(cudaMemsetAsync(ctx->attn_ticket, 0, sizeof(unsigned), ctx->stream));
        ctx->mk_bar_base = 0;
        ctx->attn_ticket_base = 0;
        return fail(ctx, SPARSK_ETIMEOUT, "a bounded in-kernel wait ran out");
    }
    if (status & ST_BAD_TOKEN) return fail(ctx, SPARSK_EINVAL, "a token id was outside the vocabulary (clamped)");
    return SPARSK_OK;
}

extern "C" int sparsk_check(sparsk_ctx *ctx)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    return read_status(ctx);
}

extern "C" int sparsk_kernel_time_by_class(sparsk_ctx *ctx, double *total_ms, int64_t *n_launches)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (!total_ms || !n_launches) return fail(ctx, SPARSK_EINVAL, "kernel_time_by_class: NULL output");
    CU(cudaStreamSynchronize(ctx->stream));
    for (int k = 0; k < 8; k++) {
        total_ms[k] = 0.0;
        n_launches[k] = 0;
    }
    for (size_t i = 0; i + 1 < ctx->tev_used; i += 2) {
        float ms = 0.f;
        CU(cudaEventElapsedTime(&ms, ctx->tev[i], ctx->tev[i + 1]));
        const int k = ctx->tev_class[i / 2] & 7;
        total_ms[k] += ms;
        n_launches[k]++;
    }
    return SPARSK_OK;
}

extern "C" int sparsk_phase_trace(sparsk_ctx *ctx, int64_t *out_ns, int32_t capacity)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (!out_ns || capacity < 0) return fail(ctx, SPARSK_EINVAL, "phase_trace: bad arguments");
    const int n = std::min<int>(capacity, ctx->mk_trace_n);
    if (n > 0) CU(cudaMemcpyAsync(out_ns, ctx->mk_trace, sizeof(int64_t) * n, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    return n;
}

extern "C" int sparsk_reset_slot(sparsk_ctx *ctx, int32_t slot) { return sparsk_set_len(ctx, slot, 0); }

extern "C" int sparsk_set_len(sparsk_ctx *ctx, int32_t slot, int32_t len)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (slot < 0 || slot >= ctx->dm.max_seqs || len < 0 || len > ctx->dm.max_seq_len)
        return fail(ctx, SPARSK_EINVAL, "set_len: slot %d / len %d out of range", slot, len);
    CU(launch(ctx, set_int_kernel, dim3(1), dim3(1), 0, ctx->kv_len + slot, (int)len));
    CU(launch(ctx, set_int_kernel, dim3(1), dim3(1), 0, ctx->pend_cnt + slot, 0));
    ctx->h_len[slot] = len;
    ctx->h_pend[slot] = 0;
    ctx->h_fill[slot].clear();
    return SPARSK_OK;
}

extern "C" int sparsk_slot_state(const sparsk_ctx *ctx, int32_t slot, int32_t *len, int32_t *pending)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (slot < 0 || slot >= ctx->dm.max_seqs) return SPARSK_EINVAL;
    if (len) *len = ctx->h_len[slot];
    if (pending) *pending = ctx->h_pend[slot];
    return SPARSK_OK;
}

static int kv_io(sparsk_ctx *ctx, int32_t slot, int32_t layer, int32_t first_pos, int32_t n, void *k, void *v, int to_cache)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    const sparsk_dims &d = ctx->dm;
    if (slot < 0 || slot >= d.max_seqs || layer < 1 || layer > d.n_layers || first_pos < 0 || n < 0 ||
        (long)first_pos + n > d.max_seq_len || !k || !v)
        return fail(ctx, SPARSK_EINVAL, "kv import/export: argument out of range");
    if (n == 0) return SPARSK_OK;
    const size_t per_slot = (size_t)d.n_kv_heads * d.max_seq_len * d.head_dim;
    const size_t off = ((size_t)(layer - 1) * d.max_seqs + slot) * per_slot;
    const size_t total = (size_t)n * d.n_kv_heads * d.head_dim;
    const int blocks = (int)std::min<size_t>((total + 255) / 256, 4096);
    CU(launch(ctx, kv_copy_kernel, dim3(blocks), dim3(256), 0, ctx->kcache + off, ctx->vcache + off, (kv_t *)k,
              (kv_t *)v, (int)first_pos, (int)n, d.n_kv_heads, d.head_dim, d.max_seq_len, to_cache));
    return SPARSK_OK;
}
extern "C" int sparsk_import_kv(sparsk_ctx *ctx, int32_t slot, int32_t layer, int32_t first_pos, int32_t n,
                                const void *k, const void *v)
{
    return kv_io(ctx, slot, layer, first_pos, n, const_cast<void *>(k), const_cast<void *>(v), 1);
}
extern "C" int sparsk_export_kv(sparsk_ctx *ctx, int32_t slot, int32_t layer, int32_t first_pos, int32_t n,
                                void *k, void *v)
{
    return kv_io(ctx, slot, layer, first_pos, n, k, v, 0);
}

// --------------------------------------------------------------------------- prefill
extern "C" int sparsk_prefill(sparsk_ctx *ctx, int32_t n_seqs, const int32_t *slots, const int32_t *tokens,
                              const int32_t *offsets)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    const sparsk_dims &d = ctx->dm;
    if (n_seqs < 0 || n_seqs > d.max_seqs || (n_seqs && (!slots || !tokens || !offsets)))
        return fail(ctx, SPARSK_EINVAL, "prefill: bad arguments");
    std::vector<char> seen(d.max_seqs, 0);
    for (int i = 0; i < n_seqs; i++) {
        const int s = slots[i];
        if (s < 0 || s >= d.max_seqs || seen[s]) return fail(ctx, SPARSK_EINVAL, "prefill: slot %d invalid or repeated", s);
        seen[s] = 1;
        const long n = (long)offsets[i + 1] - offsets[i];
        if (n < 0 || offsets[i] < 0) return fail(ctx, SPARSK_EINVAL, "prefill: offsets must not decrease");
        if (ctx->h_pend[s]) return fail(ctx, SPARSK_ESTATE, "prefill: slot %d has pending positions", s);
        if (ctx->h_len[s] + n > d.max_seq_len) return fail(ctx, SPARSK_ECAPACITY, "prefill: slot %d would hold %ld > %d positions", s, ctx->h_len[s] + n, d.max_seq_len);
    }
    const int chunk = std::min(d.prefill_rows, ctx->cap_rows);
    for (int i = 0; i < n_seqs; i++) {
        const int s = slots[i];
        const int total = offsets[i + 1] - offsets[i];
        for (int done = 0; done < total; done += chunk) {
            const int n = std::min(chunk, total - done);
            const int pos0 = ctx->h_len[s];
            CU(launch(ctx, prefill_rows_kernel, dim3((n + 255) / 256), dim3(256), 0, ctx->pf_slot, ctx->pf_pos,
                      ctx->pf_grp_row0, ctx->pf_grp_nrows, s, pos0, n));
            CU(launch(ctx, set_int_kernel, dim3(1), dim3(1), 0, ctx->pf_ngrp, 1));
            CU(launch(ctx, set_int_kernel, dim3(1), dim3(1), 0, ctx->pf_nrows, n));
            CU(launch(ctx, embed_kernel, dim3(n), dim3(128), 0, tokens + offsets[i] + done, ctx->embed, ctx->h_up, n, d.d_model,
                      d.vocab_text + d.vocab_speech, ctx->sd.counts + CNT_STATUS));
            RowSet rs{ctx->pf_slot, ctx->pf_pos, ctx->pf_grp_row0, ctx->pf_grp_nrows, ctx->pf_ngrp, ctx->pf_nrows,
                      n, 1, n, pos0 + n};
            CU(run_layers(ctx, 1, d.n_layers, ctx->h_up, rs));
            CU(launch(ctx, set_int_kernel, dim3(1), dim3(1), 0, ctx->kv_len + s, pos0 + n));
            ctx->h_len[s] = pos0 + n;
        }
    }
    return SPARSK_OK;
}

// --------------------------------------------------------------------------- decode step, confidence-based exit
// The step of a context whose dims name a confidence modality (Sec. V-B, compared method 3).
// Depths are not known beforehand, so the host walks the layers in segments: a segment is a run
// of layers over one row set; it ends where a pending position joins (the layer after the one it
// has been carried to), where a scheduled sequence leaves, and after every layer from
// conf_start on while a confidence sequence is still running, because there its head is
// consulted: head, entropy kernel, copy of the entropies to the host, stream synchronisation,
// decision.  Pending positions carry the layer they have been filled to; a sequence's rows in a
// segment are the pending positions not yet carried through its first layer (always the newest
// ones: an older position has been carried at least as far as a newer one) followed by the
// current position, i.e. consecutive positions, one attention group.
static int decode_step_conf(sparsk_ctx *ctx, int32_t n, const int32_t *slots, const int32_t *token_ids,
                            const uint8_t *modality, const int32_t *counters, int32_t *next_tokens, int32_t *exit_depths)
{
    const sparsk_dims &d = ctx->dm;
    const int L = d.n_layers, e = d.exit_layer, B = d.max_seqs, cs = d.conf_start;
    const int V = d.vocab_text + d.vocab_speech, G_heads = d.n_q_heads / d.n_kv_heads;
    const SchedParams sp{L, e, d.refresh_period, d.refresh_phase, d.text_period > 0 ? d.text_period : d.refresh_period,
                         d.text_period > 0 ? d.text_phase : d.refresh_phase, d.text_exit};
    std::vector<char> seen(B, 0);
    std::vector<int> target(n), depth(n, 0);
    int max_len = 0;
    for (int i = 0; i < n; i++) {
        const int s = slots[i];
        if (s < 0 || s >= B || seen[s]) return fail(ctx, SPARSK_EINVAL, "decode_step: slot %d invalid or repeated", s);
        seen[s] = 1;
        if (modality[i] > 1) return fail(ctx, SPARSK_EINVAL, "decode_step: modality[%d]=%d", i, modality[i]);
        if (counters[i] < 0) return fail(ctx, SPARSK_EINVAL, "decode_step: counter[%d]=%d", i, counters[i]);
        if (ctx->h_len[s] + 1 > d.max_seq_len) return fail(ctx, SPARSK_ECAPACITY, "decode_step: slot %d is full (%d positions)", s, ctx->h_len[s]);
        const bool by_conf = (d.conf_modalities >> (modality[i] ? 1 : 0)) & 1;
        target[i] = by_conf ? 0 : scheduled_depth(modality[i], counters[i], sp);
        if (target[i] != L && (int)ctx->h_fill[s].size() + 1 > d.max_pending)
            return fail(ctx, SPARSK_ECAPACITY, "decode_step: slot %d may hold %d pending positions (max_pending %d)", s,
                        (int)ctx->h_fill[s].size() + 1, d.max_pending);
        if (target[i] && (!ctx->head_norm[target[i] - 1] || !ctx->head_proj[target[i] - 1]))
            return fail(ctx, SPARSK_ENOHEAD, "decode_step: layer %d has no exit head", target[i]);
        max_len = std::max(max_len, ctx->h_len[s] + 1);
    }
    // ---- stage the host arrays; latch tokens; embed
    const int ring = ctx->stage_next;
    ctx->stage_next = (ring + 1) % STAGE_RING;
    CU(cudaEventSynchronize(ctx->stage_ev[ring]));
    int *st = ctx->stage_host[ring];
    for (int i = 0; i < n; i++) {
        st[i] = slots[i];
        st[n + i] = modality[i];
        st[2 * n + i] = counters[i];
    }
    CU(cudaMemcpyAsync(ctx->staged, st, sizeof(int) * 3 * n, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaEventRecord(ctx->stage_ev[ring], ctx->stream));
    CU(launch(ctx, schedule_kernel, dim3((n + 127) / 128), dim3(128), 0, ctx->sd, (int)n, (const int *)ctx->staged,
              (const int *)token_ids, V, sp));
    // the lower-row arrays (positions, one-row groups); "e = L" keeps every head on the lower rows
    CU(launch(ctx, compact_kernel, dim3(1), dim3(1024), 0, ctx->sd, (int)n, (const int *)ctx->kv_len,
              (const int *)ctx->pend_cnt, L, L, B));
    CU(launch(ctx, embed_kernel, dim3(n), dim3(128), 0, (const int *)ctx->sd.token, ctx->embed, ctx->h_lo, (int)n, d.d_model,
              V, ctx->sd.counts + CNT_STATUS));
    if (ctx->dbg_logits) {
        const size_t cnt = (size_t)n * V;
        CU(launch(ctx, fill_kernel, dim3((unsigned)std::min<size_t>((cnt + 255) / 256, 2048)), dim3(256), 0, ctx->dbg_logits, cnt, -INFINITY));
    }
    const int R = ctx->cap_rows;
    size_t arena = 0;  // ints of the pinned arena used so far in this step
    auto region = [&](size_t ints) -> int * {
        if (arena + ints > ctx->conf_host_ints) return nullptr;
        int *p = ctx->conf_host + arena;
        arena += ints;
        return p;
    };
    // heads of `layer` for the listed sequences (indices into the step), text and speech apart
    auto heads = [&](int layer, const std::vector<int> &who) -> int {
        for (int mod = 0; mod < 2; mod++) {
            std::vector<int> rows;
            for (int i : who)
                if ((modality[i] ? 1 : 0) == mod) rows.push_back(i);
            if (rows.empty()) continue;
            int *hb = region(rows.size());
            if (!hb) return fail(ctx, SPARSK_ECAPACITY, "decode_step: staging arena exhausted");
            std::copy(rows.begin(), rows.end(), hb);
            CU(cudaMemcpyAsync(ctx->sd.list_row + (size_t)mod * B, hb, sizeof(int) * rows.size(), cudaMemcpyHostToDevice, ctx->stream));
            CU(cudaMemcpyAsync(ctx->sd.list_seq + (size_t)mod * B, hb, sizeof(int) * rows.size(), cudaMemcpyHostToDevice, ctx->stream));
            CU(launch(ctx, clear_keys_kernel, dim3(((int)rows.size() + 127) / 128), dim3(128), 0, ctx->sd.argmax,
                      (const int *)(ctx->sd.list_row + (size_t)mod * B), (int)rows.size()));
            CU(run_head(ctx, layer, ctx->h_lo, mod, (int)rows.size()));
        }
        return SPARSK_OK;
    };
    auto leave = [&](int i, int at) -> int {   // sequence i leaves at layer `at`
        const int s = slots[i];
        depth[i] = at;
        std::vector<int> &fill = ctx->h_fill[s];
        if (at == L) {
            fill.clear();
        } else {
            CU(cudaMemcpyAsync(ctx->pend_h + ((size_t)s * d.max_pending + fill.size()) * d.d_model, ctx->h_lo + (size_t)i * d.d_model,
                               sizeof(float) * d.d_model, cudaMemcpyDeviceToDevice, ctx->stream));
            fill.push_back(at);
        }
        return SPARSK_OK;
    };

    std::vector<int> active(n);
    for (int i = 0; i < n; i++) active[i] = i;
    ctx->conf_trace.assign((size_t)n * L, -1.f);
    int l = 1;
    while (!active.empty()) {
        // ---- where this segment ends
        int seg_end = L;
        for (int i : active) {
            seg_end = std::min(seg_end, target[i] ? target[i] : std::max(l, cs));
            for (int f : ctx->h_fill[slots[i]])
                if (f >= l) seg_end = std::min(seg_end, f);
        }
        // ---- its rows
        struct Row { int slot, pos, src, seq; };
        std::vector<Row> rows;
        std::vector<int> g_row0, g_nrows;
        int max_grp = 1, n_big = 0, seg_len = 0;
        for (int i : active) {
            const int s = slots[i];
            const std::vector<int> &fill = ctx->h_fill[s];
            const int P = (int)fill.size();
            int j0 = 0;
            while (j0 < P && fill[j0] >= l) j0++;   // carried through layer l already
            g_row0.push_back((int)rows.size());
            g_nrows.push_back(P - j0 + 1);
            for (int j = j0; j < P; j++) rows.push_back({s, ctx->h_len[s] - P + j, j, i});
            rows.push_back({s, ctx->h_len[s], -1, i});
            max_grp = std::max(max_grp, P - j0 + 1);
            n_big += (P - j0 + 1) * G_heads >= ctx->attn_tc_min_q;
            seg_len = std::max(seg_len, ctx->h_len[s] + 1);
        }
        const int m = (int)rows.size(), ng = (int)active.size();
        if (m > R) return fail(ctx, SPARSK_ECAPACITY, "decode_step: %d rows exceed capacity %d", m, R);
        if (m == n && ng == n) {
            // nothing but the step's own positions, in order: the lower rows as they stand
            RowSet lo{ctx->sd.slot, ctx->sd.lo_pos, ctx->sd.lo_grp_row0, ctx->sd.lo_grp_nrows, ctx->sd.counts + CNT_NSEQ,
                      ctx->sd.counts + CNT_NSEQ, n, n, 1, seg_len};
            CU(run_layers(ctx, l, seg_end, ctx->h_lo, lo));
        } else {
            int *hb = region(4 * (size_t)R + 2 * (size_t)B + 2);
            if (!hb) return fail(ctx, SPARSK_ECAPACITY, "decode_step: staging arena exhausted");
            int *h_slot = hb, *h_pos = hb + R, *h_src = hb + 2 * R, *h_seq = hb + 3 * R, *h_g0 = hb + 4 * R, *h_gn = h_g0 + B,
                *h_cnt = h_gn + B;
            for (int k = 0; k < m; k++) {
                h_slot[k] = rows[k].slot; h_pos[k] = rows[k].pos; h_src[k] = rows[k].src; h_seq[k] = rows[k].seq;
            }
            for (int k = 0; k < ng; k++) {
                h_g0[k] = g_row0[k];
                h_gn[k] = g_nrows[k];
            }
            h_cnt[0] = ng;
            h_cnt[1] = m;
            int *dv = ctx->conf_rows_dev;
            CU(cudaMemcpyAsync(dv, hb, sizeof(int) * (4 * (size_t)R + 2 * (size_t)B + 2), cudaMemcpyHostToDevice, ctx->stream));
            int *d_slot = dv, *d_pos = dv + R, *d_src = dv + 2 * R, *d_seq = dv + 3 * R, *d_g0 = dv + 4 * R, *d_gn = d_g0 + B,
                *d_cnt = d_gn + B;
            CU(launch(ctx, rows_move_kernel, dim3(m), dim3(128), 0, ctx->h_up, ctx->h_lo, ctx->pend_h, (const int *)d_slot,
                      (const int *)d_seq, (const int *)d_src, m, d.d_model, d.max_pending, 1));
            RowSet up{d_slot, d_pos, d_g0, d_gn, d_cnt, d_cnt + 1, m, ng, max_grp, seg_len, n_big};
            CU(run_layers(ctx, l, seg_end, ctx->h_up, up));
            CU(launch(ctx, rows_move_kernel, dim3(m), dim3(128), 0, ctx->h_up, ctx->h_lo, ctx->pend_h, (const int *)d_slot,
                      (const int *)d_seq, (const int *)d_src, m, d.d_model, d.max_pending, 0));
        }
        for (int i : active)   // the pending positions that took part have been carried to seg_end
            for (int &f : ctx->h_fill[slots[i]])
                if (f < seg_end) f = seg_end;
        // ---- who leaves after layer seg_end
        std::vector<int> leaving, asking;
        for (int i : active) {
            if (seg_end == L || target[i] == seg_end) leaving.push_back(i);
            else if (!target[i] && seg_end >= cs) asking.push_back(i);
        }
        if (!leaving.empty()) {
            const int rc = heads(seg_end, leaving);
            if (rc != SPARSK_OK) return rc;
        }
        if (!asking.empty()) {
            int rc = heads(seg_end, asking);
            if (rc != SPARSK_OK) return rc;
            int *hb = region(2 * asking.size());
            if (!hb) return fail(ctx, SPARSK_ECAPACITY, "decode_step: staging arena exhausted");
            for (size_t k = 0; k < asking.size(); k++) {
                hb[k] = asking[k];
                hb[asking.size() + k] = modality[asking[k]] ? 1 : 0;
            }
            CU(cudaMemcpyAsync(ctx->conf_list_dev, hb, sizeof(int) * 2 * asking.size(), cudaMemcpyHostToDevice, ctx->stream));
            CU(launch(ctx, entropy_kernel, dim3((unsigned)asking.size()), dim3(1024), 0, (const float *)head_logits(ctx),
                      (const int *)ctx->conf_list_dev, (const int *)(ctx->conf_list_dev + asking.size()), (int)asking.size(), V,
                      d.vocab_text, ctx->conf_ent_dev));
            CU(cudaMemcpyAsync(ctx->conf_ent_host, ctx->conf_ent_dev, sizeof(float) * asking.size(), cudaMemcpyDeviceToHost, ctx->stream));
            CU(cudaStreamSynchronize(ctx->stream));
            for (size_t k = 0; k < asking.size(); k++) {
                ctx->conf_trace[(size_t)asking[k] * L + seg_end] = ctx->conf_ent_host[k];
                if (ctx->conf_ent_host[k] < d.conf_threshold) leaving.push_back(asking[k]);
            }
        }
        for (int i : leaving) {
            const int rc = leave(i, seg_end);
            if (rc != SPARSK_OK) return rc;
            active.erase(std::find(active.begin(), active.end(), i));
        }
        l = seg_end + 1;
    }
    // ---- outputs and state
    int *hb = region(n);
    if (!hb) return fail(ctx, SPARSK_ECAPACITY, "decode_step: staging arena exhausted");
    std::copy(depth.begin(), depth.end(), hb);
    CU(cudaMemcpyAsync(ctx->sd.depth, hb, sizeof(int) * n, cudaMemcpyHostToDevice, ctx->stream));
    if (ctx->dbg_hidden)
        CU(launch(ctx, debug_hidden_kernel, dim3(n), dim3(128), 0, ctx->sd, (const float *)ctx->h_lo,
                  (const float *)ctx->h_up, ctx->dbg_hidden, (int)n, d.d_model));
    CU(launch(ctx, finish_kernel, dim3((n + 127) / 128), dim3(128), 0, ctx->sd, (int)n, ctx->kv_len, ctx->pend_cnt,
              next_tokens, exit_depths, L));
    for (int i = 0; i < n; i++) {
        ctx->h_len[slots[i]] += 1;
        ctx->h_pend[slots[i]] = (int)ctx->h_fill[slots[i]].size();
    }
    CU(cudaStreamSynchronize(ctx->stream));  // the pinned arena is free again
    return SPARSK_OK;
}

// --------------------------------------------------------------------------- decode step
extern "C" int sparsk_decode_step(sparsk_ctx *ctx, int32_t n, const int32_t *slots, const int32_t *token_ids,
                                  const uint8_t *modality, const int32_t *counters, int32_t *next_tokens,
                                  int32_t *exit_depths)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    const sparsk_dims &d = ctx->dm;
    const int L = d.n_layers, e = d.exit_layer, B = d.max_seqs;
    const SchedParams sp{L, e, d.refresh_period, d.refresh_phase, d.text_period > 0 ? d.text_period : d.refresh_period,
                         d.text_period > 0 ? d.text_phase : d.refresh_phase, d.text_exit};
    if (n < 1 || n > B || !slots || !token_ids || !modality || !counters || !next_tokens || !exit_depths)
        return fail(ctx, SPARSK_EINVAL, "decode_step: bad arguments (n=%d)", n);
    if (d.conf_modalities) return decode_step_conf(ctx, n, slots, token_ids, modality, counters, next_tokens, exit_depths);
    // ---- host mirror of the schedule: validates, and sizes the launches
    std::vector<char> seen(B, 0);
    int n_list[4] = {0, 0, 0, 0};
    int m_up = 0, n_grp = 0, max_grp = 1, max_len_lo = 0, max_len_up = 0, n_big = 0;
    long sum_len_lo = 0, sum_len_up = 0;
    const int G_heads = d.n_q_heads / d.n_kv_heads;
    for (int i = 0; i < n; i++) {
        const int s = slots[i];
        if (s < 0 || s >= B || seen[s]) return fail(ctx, SPARSK_EINVAL, "decode_step: slot %d invalid or repeated", s);
        seen[s] = 1;
        if (modality[i] > 1) return fail(ctx, SPARSK_EINVAL, "decode_step: modality[%d]=%d", i, modality[i]);
        if (counters[i] < 0) return fail(ctx, SPARSK_EINVAL, "decode_step: counter[%d]=%d", i, counters[i]);
        if (ctx->h_len[s] + 1 > d.max_seq_len) return fail(ctx, SPARSK_ECAPACITY, "decode_step: slot %d is full (%d positions)", s, ctx->h_len[s]);
        const int depth = scheduled_depth(modality[i], counters[i], sp);
        const bool full = depth == L;
        if (!full && ctx->h_pend[s] + 1 > d.max_pending)
            return fail(ctx, SPARSK_ECAPACITY, "decode_step: slot %d would hold %d pending positions (max_pending %d)", s, ctx->h_pend[s] + 1, d.max_pending);
        n_list[(full ? 2 : 0) + (modality[i] ? 1 : 0)]++;
        max_len_lo = std::max(max_len_lo, ctx->h_len[s] + 1);
        sum_len_lo += ctx->h_len[s] + 1;
        if (full && e < L) {
            sum_len_up += ctx->h_len[s] + 1;
            m_up += ctx->h_pend[s] + 1;
            n_grp++;
            max_grp = std::max(max_grp, ctx->h_pend[s] + 1);
            n_big += (ctx->h_pend[s] + 1) * G_heads >= ctx->attn_tc_min_q;
            max_len_up = std::max(max_len_up, ctx->h_len[s] + 1);
        }
    }
    if ((n_list[0] + n_list[1]) && (!ctx->head_norm[e - 1] || !ctx->head_proj[e - 1]))
        return fail(ctx, SPARSK_ENOHEAD, "decode_step: layer %d has no exit head", e);
    if (m_up > ctx->cap_rows) return fail(ctx, SPARSK_ECAPACITY, "decode_step: %d upper rows exceed capacity %d", m_up, ctx->cap_rows);

    // ---- stage the host arrays
    const int ring = ctx->stage_next;
    ctx->stage_next = (ring + 1) % STAGE_RING;
    CU(cudaEventSynchronize(ctx->stage_ev[ring]));
    int *st = ctx->stage_host[ring];
    for (int i = 0; i < n; i++) {
        st[i] = slots[i];
        st[n + i] = modality[i];
        st[2 * n + i] = counters[i];
    }
    CU(cudaMemcpyAsync(ctx->staged, st, sizeof(int) * 3 * n, cudaMemcpyHostToDevice, ctx->stream));
    CU(cudaEventRecord(ctx->stage_ev[ring], ctx->stream));

    // ---- schedule, compaction, embedding
    const int V = d.vocab_text + d.vocab_speech;
    CU(launch(ctx, schedule_kernel, dim3((n + 127) / 128), dim3(128), 0, ctx->sd, (int)n, (const int *)ctx->staged,
              (const int *)token_ids, V, sp));
    CU(launch(ctx, compact_kernel, dim3(1), dim3(1024), 0, ctx->sd, (int)n, (const int *)ctx->kv_len,
              (const int *)ctx->pend_cnt, L, e, B));
    CU(launch(ctx, embed_kernel, dim3(n), dim3(128), 0, (const int *)ctx->sd.token, ctx->embed, ctx->h_lo, (int)n, d.d_model,
              V, ctx->sd.counts + CNT_STATUS));
    if (ctx->dbg_logits) {
        const size_t cnt = (size_t)n * V;
        CU(launch(ctx, fill_kernel, dim3((unsigned)std::min<size_t>((cnt + 255) / 256, 2048)), dim3(256), 0, ctx->dbg_logits, cnt, -INFINITY));
    }
    // ---- lower pass: layers 1..e over all sequences
    RowSet lo{ctx->sd.slot, ctx->sd.lo_pos, ctx->sd.lo_grp_row0, ctx->sd.lo_grp_nrows, ctx->sd.counts + CNT_NSEQ,
              ctx->sd.counts + CNT_NSEQ, n, n, 1, max_len_lo};
    lo.sum_len = sum_len_lo;
    CU(run_layers(ctx, 1, e, ctx->h_lo, lo));
    // ---- early exits: keep h^(e), read the token from g_e
    if (n_list[0] + n_list[1]) {
        CU(launch(ctx, stash_kernel, dim3(n), dim3(128), 0, ctx->sd, (const float *)ctx->h_lo, ctx->pend_h,
                  (const int *)ctx->pend_cnt, (int)n, d.d_model, L, d.max_pending));
        for (int l = 0; l < 2; l++)
            if (n_list[l]) CU(run_head(ctx, e, ctx->h_lo, l, n_list[l]));
    }
    // ---- upper pass: pending and current positions of full-depth sequences through e+1..L
    const float *h_full = ctx->h_lo;
    if (m_up) {
        CU(launch(ctx, gather_upper_kernel, dim3(m_up), dim3(128), 0, ctx->sd, (const float *)ctx->h_lo,
                  (const float *)ctx->pend_h, ctx->h_up, d.d_model, d.max_pending));
        RowSet up{ctx->sd.up_slot, ctx->sd.up_pos, ctx->sd.up_grp_row0, ctx->sd.up_grp_nrows, ctx->sd.counts + CNT_NGRP,
                  ctx->sd.counts + CNT_MUP, m_up, n_grp, max_grp, max_len_up, n_big};
        up.sum_len = sum_len_up;
        // Layer L gives the pending rows nothing but their K/V: nothing reads their h^(L).  When the
        // step has pending rows and the rest of the layer is cheaper on one row per sequence
        // (attention over long prefixes, projections with enough rows to be tensor-bound), the
        // layer's back half runs on the current rows alone.
        const int qd = d.n_q_heads * d.head_dim;
        const bool persistent = use_mega(ctx, m_up);
        const bool trim = m_up > n_grp && !persistent &&
                          (ctx->trim_last == 2 || (ctx->trim_last == 1 && use_tc(ctx, n_grp)));
        if (!trim) {
            CU(run_layers(ctx, e + 1, L, ctx->h_up, up));
        } else {
            CU(run_layers(ctx, e + 1, L - 1, ctx->h_up, up));
            ctx->route_layers[use_tc(ctx, m_up) ? 1 : 2] += 1;
            CU(run_layer_front(ctx, L, ctx->h_up, up));
            CU(launch(ctx, take_current_kernel, dim3(n_grp), dim3(256), 0, ctx->sd, (const float *)ctx->h_up,
                      (const float *)ctx->qbuf, ctx->h_last, ctx->q_last, ctx->last_slot, ctx->last_pos, d.d_model, qd));
            RowSet last{ctx->last_slot, ctx->last_pos, ctx->sd.lo_grp_row0, ctx->sd.lo_grp_nrows, ctx->sd.counts + CNT_NGRP,
                        ctx->sd.counts + CNT_NGRP, n_grp, n_grp, 1, max_len_up, 0, ctx->q_last};
            last.sum_len = sum_len_up;
            CU(run_layer_back(ctx, L, ctx->h_last, last));
            CU(launch(ctx, put_current_kernel, dim3(n_grp), dim3(256), 0, ctx->sd, (const float *)ctx->h_last, ctx->h_up,
                      d.d_model));
        }
        h_full = ctx->h_up;
    }
    for (int l = 2; l < 4; l++)
        if (n_list[l]) CU(run_head(ctx, L, h_full, l, n_list[l]));
    if (ctx->samp_uniforms) {
        // replace the arg max by a draw from the nucleus of the same logits (Sec. V-A)
        SampleArgs sa{};
        sa.logits = head_logits(ctx); sa.uniforms = ctx->samp_uniforms;
        sa.modality = ctx->sd.modality; sa.key_out = ctx->sd.argmax; sa.token_out = nullptr;
        sa.V = V; sa.Vt = d.vocab_text; sa.Vs = d.vocab_speech;
        sa.inv_temperature = 1.f / ctx->samp_temperature; sa.top_p = ctx->samp_top_p;
        const bool timed = (ctx->time_class == KC_HEAD || ctx->time_class == KC_ALL) && ctx->tev_used + 2 <= ctx->tev.size();
        if (timed) {
            ctx->tev_class[ctx->tev_used / 2] = KC_HEAD;
            cudaEventRecord(ctx->tev[ctx->tev_used++], ctx->stream);
        }
        CU(launch_nucleus_sample(sa, n, n_list[0] + n_list[2] > 0, n_list[1] + n_list[3] > 0, ctx->stream, ctx->pdl != 0,
                                 &ctx->launches));
        if (timed) cudaEventRecord(ctx->tev[ctx->tev_used++], ctx->stream);
    }
    if (ctx->dbg_hidden)
        CU(launch(ctx, debug_hidden_kernel, dim3(n), dim3(128), 0, ctx->sd, (const float *)ctx->h_lo,
                  (const float *)ctx->h_up, ctx->dbg_hidden, (int)n, d.d_model));
    CU(launch(ctx, finish_kernel, dim3((n + 127) / 128), dim3(128), 0, ctx->sd, (int)n, ctx->kv_len, ctx->pend_cnt,
              next_tokens, exit_depths, L));
    // ---- host mirror follows
    for (int i = 0; i < n; i++) {
        const int s = slots[i];
        const int depth = scheduled_depth(modality[i], counters[i], sp);
        ctx->h_len[s] += 1;
        ctx->h_pend[s] = (depth == L) ? 0 : ctx->h_pend[s] + 1;
    }
    return SPARSK_OK;
}

extern "C" int sparsk_decode_step_host(sparsk_ctx *ctx, int32_t n, const int32_t *slots, const int32_t *token_ids,
                                       const uint8_t *modality, const int32_t *counters, int32_t *next_tokens,
                                       int32_t *exit_depths)
{
    if (!good(ctx)) return SPARSK_ESTATE;
    if (n < 1 || n > ctx->dm.max_seqs || !token_ids || !next_tokens || !exit_depths)
        return fail(ctx, SPARSK_EINVAL, "decode_step_host: bad arguments (n=%d)", n);
    // the tokens are host data here, so their range is checked like every other host argument:
    // before anything is enqueued, leaving all state as it was
    const int V = ctx->dm.vocab_text + ctx->dm.vocab_speech;
    for (int i = 0; i < n; i++)
        if (token_ids[i] < 0 || token_ids[i] >= V)
            return fail(ctx, SPARSK_EINVAL, "decode_step_host: token_ids[%d]=%d is outside the vocabulary [0, %d)", i, token_ids[i], V);
    // Everything crosses the bus through one pinned buffer, so that the copies are truly
    // asynchronous and the host waits once per step (a copy to or from pageable memory makes the
    // host wait for it; three of them in a row after the step cost 30 us of idle GPU per step).
    const int B = ctx->dm.max_seqs;
    int *io = ctx->io_host;
    memcpy(io, token_ids, sizeof(int) * n);
    CU(cudaMemcpyAsync(ctx->tok_dev, io, sizeof(int) * n, cudaMemcpyHostToDevice, ctx->stream));
    const int rc = sparsk_decode_step(ctx, n, slots, ctx->tok_dev, modality, counters, ctx->out_tok_dev, ctx->out_depth_dev);
    if (rc != SPARSK_OK) return rc;
    CU(cudaMemcpyAsync(io + B, ctx->out_tok_dev, sizeof(int) * n, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaMemcpyAsync(io + 2 * B, ctx->out_depth_dev, sizeof(int) * n, cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaMemcpyAsync(io + 3 * B, ctx->sd.counts + CNT_STATUS, sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    CU(cudaStreamSynchronize(ctx->stream));
    memcpy(next_tokens, io + B, sizeof(int) * n);
    memcpy(exit_depths, io + 2 * B, sizeof(int) * n);
    return act_on_status(ctx, io[3 * B]);
}

// Stand-alone entry points for single kernels of the decode path (C ABI in include/sparsk.h).
// They run exactly the kernels a decode step runs, on caller-described inputs, so that one
// stage can be driven, checked and profiled on its own.
#include <algorithm>
#include <cstdint>

#include "../../include/sparsk.h"
#include "sparsk_attn.cuh"
#include "sparsk_sample.cuh"
#include "sparsk_step.cuh"

using namespace sparsk;

namespace {
size_t up256(size_t v) { return (v + 255) / 256 * 256; }
}  // namespace

static bool attn_args_ok(const sparsk_attn_args *a)
{
    if (!a || !a->q || !a->k_cache || !a->v_cache || !a->out || !a->row_slot || !a->row_pos || !a->grp_row0 ||
        !a->grp_nrows)
        return false;
    if (a->n_rows < 1 || a->n_groups < 1 || a->n_groups > a->n_rows || a->max_grp_rows < 1 ||
        a->max_grp_rows > a->n_rows)
        return false;
    if (a->n_q_heads < 1 || a->n_kv_heads < 1 || a->n_q_heads % a->n_kv_heads) return false;
    if (a->head_dim != 64 && a->head_dim != 128) return false;
    if (a->cache_len < 1 || a->n_slots < 1 || a->max_len < 1 || a->max_len > a->cache_len) return false;
    return true;
}

extern "C" size_t sparsk_attention_scratch_bytes(int32_t n_rows, int32_t n_q_heads, int32_t head_dim)
{
    if (n_rows < 1 || n_q_heads < 1 || (head_dim != 64 && head_dim != 128)) return 0;
    const size_t cells = (size_t)n_rows * n_q_heads * AT_MAX_SPLITS;
    return 256 + up256(cells * head_dim * sizeof(float)) + up256(cells * sizeof(float2));
}

// Shared by the entry points of this library that run the two attention kernels outside a
// context: `scratch` holds two counters, then the split partials.
int sparsk_attention_launch(const sparsk_attn_args *p, char *scratch, cudaStream_t st)
{
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
        return SPARSK_ECUDA;
    const size_t cells = (size_t)p->n_rows * p->n_q_heads * AT_MAX_SPLITS;
    int *counts = reinterpret_cast<int *>(scratch);
    AttnArgs a{};
    a.q = (const bf16 *)p->q; a.kc = (const kv_t *)p->k_cache; a.vc = (const kv_t *)p->v_cache;
    a.grp_row0 = p->grp_row0; a.grp_nrows = p->grp_nrows; a.row_slot = p->row_slot; a.row_pos = p->row_pos;
    a.n_groups = counts;
    a.part_o = reinterpret_cast<float *>(scratch + 256);
    a.part_ml = reinterpret_cast<float2 *>(scratch + 256 + up256(cells * p->head_dim * sizeof(float)));
    a.out = (bf16 *)p->out;
    a.Hq = p->n_q_heads; a.Hkv = p->n_kv_heads; a.S = p->cache_len; a.n_slots = p->n_slots; a.n_rows = p->n_rows;
    a.nq_min = 0; a.nq_max = 1 << 30;
    const int warp_ctas = n_sm * attn_warp_ctas_per_sm(p->head_dim, AW_NST);
    const AttnPlan pl = attn_plan(warp_ctas * AW_WARPS, p->n_groups, p->max_grp_rows, p->n_q_heads / p->n_kv_heads,
                                  p->n_kv_heads, p->max_len, 0);
    a.n_qblk = pl.n_qblk; a.split_len = pl.split_len; a.n_splits = pl.n_splits;
    a.max_groups = p->n_groups;
    set_int_kernel<<<1, 1, 0, st>>>(counts, p->n_groups);
    set_int_kernel<<<1, 1, 0, st>>>(counts + 1, p->n_rows);
    const long n_items = (long)p->n_groups * pl.n_qblk * p->n_kv_heads * pl.n_splits;
    const int grid = (int)std::max<long>(1, std::min<long>(warp_ctas, (n_items + AW_WARPS - 1) / AW_WARPS));
    AttnWarpFn fn;
    if (attn_warp_fn(p->head_dim, AW_NST, &fn) != cudaSuccess) return SPARSK_ECUDA;
    fn<<<grid, AW_WARPS * 32, AW_WARPS * attn_warp_bytes(p->head_dim, AW_NST), st>>>(a);
    if (p->head_dim == 128) attn_merge_kernel<128><<<dim3(p->n_rows, p->n_q_heads), 128, 0, st>>>(a, counts + 1);
    else attn_merge_kernel<64><<<dim3(p->n_rows, p->n_q_heads), 64, 0, st>>>(a, counts + 1);
    return cudaGetLastError() == cudaSuccess ? SPARSK_OK : SPARSK_ECUDA;
}

extern "C" int sparsk_attention(const sparsk_attn_args *args, void *scratch, size_t scratch_bytes, void *cuda_stream)
{
    if (!attn_args_ok(args) || !scratch || ((uintptr_t)scratch % 256)) return SPARSK_EINVAL;
    if (scratch_bytes < sparsk_attention_scratch_bytes(args->n_rows, args->n_q_heads, args->head_dim))
        return SPARSK_EINVAL;
    return sparsk_attention_launch(args, (char *)scratch, (cudaStream_t)cuda_stream);
}

extern "C" int sparsk_nucleus_sample(const float *logits, const float *uniforms, const int32_t *modality, int32_t n,
                                     int32_t vocab_text, int32_t vocab_speech, float temperature, float top_p,
                                     int32_t *tokens, void *cuda_stream)
{
    if (!logits || !uniforms || !modality || !tokens) return SPARSK_EINVAL;
    if (n < 1 || vocab_text < 1 || vocab_speech < 0 || vocab_text > SP_MAX_RANGE || vocab_speech > SP_MAX_RANGE)
        return SPARSK_EINVAL;
    if (!(temperature > 0.f) || !(temperature < INFINITY) || !(top_p > 0.f) || !(top_p <= 1.f)) return SPARSK_EINVAL;
    SampleArgs a{};
    a.logits = logits; a.uniforms = uniforms; a.modality = modality;
    a.key_out = nullptr; a.token_out = tokens;
    a.V = vocab_text + vocab_speech; a.Vt = vocab_text; a.Vs = vocab_speech;
    a.inv_temperature = 1.f / temperature; a.top_p = top_p;
    return launch_nucleus_sample(a, n, true, vocab_speech > 0, (cudaStream_t)cuda_stream, false, nullptr) == cudaSuccess
               ? SPARSK_OK
               : SPARSK_ECUDA;
}

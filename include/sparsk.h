/*
 * sparsk.h -- C ABI of the B200 (sm_100a) SPAR-K decode library.
 *
 * SPAR-K (scheduled periodic alternating early exit) decodes an interleaved
 * text/speech token stream with a stack of L transformer layers.  Text steps run
 * all L layers.  A speech step whose index c inside its chunk satisfies
 * c mod K == r runs all L layers too ("refresh"); every other speech step leaves
 * at layer e = l_EE and reads its token from that layer's own head (Sec. IV-B.1,
 * Eq. 2).  An early-exit step caches K/V of layers 1..e only, keeps h^(e) and
 * marks its position pending; the next full-depth step pushes the pending
 * positions together with its own through layers e+1..L as one causal block,
 * which fills their K/V, and clears the pending set; tokens already emitted are
 * never revised (Sec. IV-B.3, Algorithm 1).
 *
 * Every step of that path runs in hand-written CUDA kernels inside this library.
 * There is no CPU fallback.  The library never calls cudaMalloc on the step path:
 * all device memory is a caller-supplied workspace.
 *
 * Conventions
 *   - "device" / "host" in a comment says where the pointer must live.
 *   - All weights are bfloat16, row-major [out_features, in_features], BORROWED:
 *     the caller keeps them alive until sparsk_destroy.
 *   - Token ids [0, vocab_text) are text, [vocab_text, vocab_text+vocab_speech)
 *     are speech.
 *   - Calls enqueue work on the stream given at create and return without
 *     synchronising unless stated.  Outputs are valid once the stream has been
 *     synchronised.
 *   - Return value 0 is success, negative values are the SPARSK_E* codes.  Every
 *     error that can be found from host-side arguments is found before anything
 *     is launched, and leaves all state unchanged.  Nothing aborts or traps.
 */
#ifndef SPARSK_H
#define SPARSK_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define SPARSK_OK 0
#define SPARSK_EINVAL (-1)    /* bad dims, NULL pointer, value out of range, duplicate slot   */
#define SPARSK_ECAPACITY (-2) /* a sequence would exceed max_seq_len or max_pending           */
#define SPARSK_ENOHEAD (-3)   /* the step needs an exit head whose pointers are NULL          */
#define SPARSK_ECUDA (-4)     /* a CUDA call failed; text in sparsk_last_error                */
#define SPARSK_ESTATE (-5)    /* slot in the wrong state for the call / not a context         */
#define SPARSK_ETIMEOUT (-6)  /* a bounded in-kernel wait ran out (reported by the next call) */

typedef struct sparsk_ctx sparsk_ctx; /* opaque */

/* Model and schedule description (Sec. III for L and d; Sec. IV-B.1 for e, K, r). */
typedef struct {
    int32_t n_layers;       /* L */
    int32_t d_model;        /* d, multiple of 8 */
    int32_t n_q_heads;      /* H_q, multiple of n_kv_heads */
    int32_t n_kv_heads;     /* H_kv */
    int32_t head_dim;       /* 64 or 128 */
    int32_t d_ffn;          /* F, multiple of 8 */
    int32_t vocab_text;     /* V_t */
    int32_t vocab_speech;   /* V_s */
    float rms_eps;
    float rope_base;
    int32_t exit_layer;     /* e in 1..L; e == L disables early exit */
    int32_t refresh_period; /* K >= 1; K == 1 makes every step full depth */
    int32_t refresh_phase;  /* r in [0, K): in-chunk index c is full depth iff c % K == r */
    int32_t text_exit;      /* 0: text steps always run L layers (the paper's main rows);
                               1: text steps follow the same (K, r, e) rule as speech steps;
                               2: only text steps follow it and speech steps always run L
                                  layers (Sec. V-E, row G10) */
    int32_t max_seqs;       /* number of sequence slots */
    int32_t max_seq_len;    /* positions per slot */
    int32_t max_pending;    /* pending positions per slot; >= K-1 for the periodic schedule */
    int32_t prefill_rows;   /* rows per prefill pass (0 = default) */
    int32_t text_period;    /* K of text steps when they follow the rule (text_exit 1 or 2); 0 = the
                               same K and r as speech steps.  Sec. V-E: the two modalities may need
                               different policies */
    int32_t text_phase;     /* r of text steps, in [0, text_period) */
    /* Confidence-based early exit, the compared method of Sec. V-B (thresholds of Sec. VI: 0.1
     * for the 28-layer backbone, 0.5 for the 40-layer one).  Steps that emit a token of a
     * modality in conf_modalities (bit 0 text, bit 1 speech; 0 = off) ignore the schedule: after
     * every layer l in [conf_start, L) the head g_l is applied to the position's hidden state and
     * the step leaves at the first layer whose prediction, over the ids of the modality, has an
     * entropy (natural logarithm) below conf_threshold; otherwise it runs all L layers.  Such a
     * position is pending exactly like a scheduled early exit: later steps carry it upwards as
     * far as they go themselves.  Needs heads for the layers conf_start .. L.  A context in
     * this mode synchronises its stream inside every decode step (the host learns each depth
     * when the kernels do) and does not offer nucleus sampling. */
    int32_t conf_modalities;
    int32_t conf_start;
    float conf_threshold;
} sparsk_dims;

/* All pointers are DEVICE pointers to bfloat16 data; the arrays of pointers themselves
 * are HOST arrays of length n_layers.  head_norm[l-1] / head_proj[l-1] are the head g_l of
 * layer l (Eq. 2; g_L is the ordinary LM head of Eq. 1) and may be NULL for layers that are
 * never used as an exit. */
typedef struct {
    const void *embed;             /* [V_t+V_s, d] */
    const void *const *attn_norm;  /* [d]          */
    const void *const *wq;         /* [H_q*hd, d]  */
    const void *const *wk;         /* [H_kv*hd, d] */
    const void *const *wv;         /* [H_kv*hd, d] */
    const void *const *wo;         /* [d, H_q*hd]  */
    const void *const *mlp_norm;   /* [d]          */
    const void *const *w_gate;     /* [F, d]       */
    const void *const *w_up;       /* [F, d]       */
    const void *const *w_down;     /* [d, F]       */
    const void *const *head_norm;  /* [d] or NULL  */
    const void *const *head_proj;  /* [V_t+V_s, d] or NULL */
} sparsk_weights;

/* Bytes of device workspace sparsk_create needs for these dims; 0 if the dims are invalid.
 * No counterpart in the paper (memory management).  The workspace holds the KV cache
 * ([L][slot][H_kv][max_seq_len][hd] fp16, keys and values),
 * the pending store ([slot][max_pending][d] fp32), per-slot lengths, the step descriptor,
 * activation buffers, split-KV scratch and the rotary table. */
size_t sparsk_workspace_bytes(const sparsk_dims *dims /*host*/);

/* Build a context.  `workspace` (device, 256-byte aligned, >= sparsk_workspace_bytes) and the
 * weights stay owned by the caller.  `cuda_stream` is a cudaStream_t (NULL = default stream).
 * Synchronises the stream once (table upload).  Sec. III / IV-B define what is being set up. */
int sparsk_create(const sparsk_dims *dims /*host*/, const sparsk_weights *weights /*host*/,
                  void *workspace /*device*/, size_t workspace_bytes, void *cuda_stream,
                  sparsk_ctx **out /*host*/);

/* Ingest prompt tokens at full depth: K/V of every layer is written for every token, nothing
 * is emitted, pending sets stay empty (the standard-decoding state of Sec. III).  `slots`
 * [n_seqs] host, distinct; `tokens` device int32, the prompts concatenated; `offsets`
 * [n_seqs+1] host.  Appends to whatever the slot already holds. */
int sparsk_prefill(sparsk_ctx *ctx, int32_t n_seqs, const int32_t *slots /*host*/,
                   const int32_t *tokens /*device*/, const int32_t *offsets /*host*/);

/* One decoding step for n_seqs sequences (one iteration of Algorithm 1's loop, for text and
 * speech alike).  token_ids[i]: input token of sequence i (the token emitted by its previous
 * step, or the last prompt token).  modality[i]: 0 text / 1 speech, the modality of the token
 * this step EMITS; the argmax is restricted to that id range (lowest id on ties).
 * speech_counters[i]: index c of that token inside its chunk.  Outputs: next_tokens[i] and
 * exit_depths[i] (e or L).  Host arrays are read before the call returns.  The token ids live
 * on the device, so the host cannot check them: an id outside [0, V_t+V_s) is clamped into the
 * vocabulary by the kernels, the step runs and advances its slots, and the next sparsk_check
 * reports SPARSK_EINVAL. */
int sparsk_decode_step(sparsk_ctx *ctx, int32_t n_seqs, const int32_t *slots /*host*/,
                       const int32_t *token_ids /*device [n]*/, const uint8_t *modality /*host [n]*/,
                       const int32_t *speech_counters /*host [n]*/,
                       int32_t *next_tokens /*device [n]*/, int32_t *exit_depths /*device [n]*/);

/* The same iteration of Algorithm 1 with HOST token and result buffers: copies token_ids to the
 * device, runs the step, copies both results back and synchronises the stream.  This is the call
 * a host-side generation loop makes when it consumes every token as it is produced.  Token ids
 * outside [0, V_t+V_s) are refused with SPARSK_EINVAL before anything is launched (state
 * unchanged).  If a bounded in-kernel wait ran out during the step the call returns
 * SPARSK_ETIMEOUT once, the kernels' barrier state is reset, and the slots that took part hold
 * an incomplete step: reset them (sparsk_reset_slot) before using them again. */
int sparsk_decode_step_host(sparsk_ctx *ctx, int32_t n_seqs, const int32_t *slots /*host*/,
                            const int32_t *token_ids /*host [n]*/, const uint8_t *modality /*host*/,
                            const int32_t *speech_counters /*host*/,
                            int32_t *next_tokens /*host [n]*/, int32_t *exit_depths /*host [n]*/);

/* Forget a slot: length 0, pending set empty (the state Algorithm 1 starts a sequence from).
 * No counterpart in the paper beyond that: slot management. */
int sparsk_reset_slot(sparsk_ctx *ctx, int32_t slot);

/* Load / read cache contents of one layer (1-based) of a slot: n positions starting at
 * first_pos, keys already rotated, layout [n][H_kv*hd] fp16 (IEEE half, the cache's own element
 * type: weights are bf16, but the cache keeps 11 significant bits), device pointers.  set_len declares
 * that positions [0, len) are complete at every layer (pending set empty).  These let a caller
 * restore a saved prefix, and let tests inspect the KV invariant of Sec. IV-B.3. */
int sparsk_import_kv(sparsk_ctx *ctx, int32_t slot, int32_t layer, int32_t first_pos, int32_t n,
                     const void *k /*device*/, const void *v /*device*/);
int sparsk_export_kv(sparsk_ctx *ctx, int32_t slot, int32_t layer, int32_t first_pos, int32_t n,
                     void *k /*device*/, void *v /*device*/);
int sparsk_set_len(sparsk_ctx *ctx, int32_t slot, int32_t len);
/* Host view of a slot: positions held and size of the pending set P of Algorithm 1 (no device
 * access).  No counterpart in the paper: inspection only. */
int sparsk_slot_state(const sparsk_ctx *ctx, int32_t slot, int32_t *len /*host*/,
                      int32_t *pending /*host*/);

/* Parity hooks.  While non-NULL, every decode step also writes, for sequence i of the step,
 * the hidden state its head read (exit_hidden [n, d] fp32: h^(e) or h^(L), the argument of g_e
 * in Eq. 2 or of g_L in Eq. 1) and its logits (exit_logits [n, V_t+V_s] fp32, -inf outside the
 * modality's id range).  Device pointers, caller-owned, registered BEFORE the steps they are to
 * observe: the heads write logits only while a buffer is registered, nothing of a step is kept
 * otherwise. */
int sparsk_set_debug(sparsk_ctx *ctx, float *exit_hidden /*device or NULL*/,
                     float *exit_logits /*device or NULL*/);

/* Tuning knobs, by name (no counterpart in the paper: implementation choices): "gemm_min_rows" (row count from which the tcgen05 path is used; a
 * large value keeps everything on the GEMV path), "mega" (0/1: run passes of up to
 * four rows as one persistent kernel per layer range; default 1), "mega_max_rows" (1..4: the
 * largest pass that kernel takes; default 4. Passes of three and four rows use its tensor-core
 * inner loop, which needs d_model, d_ffn and n_heads * head_dim to be multiples of 64; other
 * shapes stop at two rows), "gemm_kb" (1: one 64-element block of the inner
 * dimension per TMA copy instead of two; 0 = automatic), "attn_split" (positions
 * per KV split), "attn_dynamic" (0/1: the attention kernel's warps draw their work items from a
 * counter as they finish instead of taking every n-th one; default 1), "attn_ctas" (CTAs of that
 * kernel; 0 = as many as fit the SMs), "attn_tma" (0/1: its K/V tiles arrive as TMA boxes with the
 * 128-byte swizzle instead of per-lane 16-byte copies; default 1), "attn_stages" (2 or 3 tiles per
 * warp's ring), "pdl" (0/1, programmatic dependent launch between the kernels of a step; default 1),
 * "gemv_ks" / "gemv_r" (override the GEMV team width / rows per group; 0 = automatic),
 * "trim_last_layer" (0/1/2: in a full-depth step, pending rows leave layer L after its K/V
 * projection, since Algorithm 1's full-depth branch reads h^(L) of the current position only; 1,
 * the default, does so when the remaining rows still fill the tensor-core path, 2 whenever a step
 * has pending rows, 0 never; results are identical),
 * "time_kernel" (see sparsk_kernel_time), "inject_barrier_timeout" (test hook, 1: the next launch
 * of the persistent kernel is given a grid-barrier count that no CTA can reach, so its bounded
 * wait runs out after about two seconds, the kernel returns and the step reports
 * SPARSK_ETIMEOUT; nothing faults or hangs).  Returns SPARSK_EINVAL for an unknown name or value. */
int sparsk_set_option(sparsk_ctx *ctx, const char *name /*host*/, int64_t value);

/* Nucleus sampling (Sec. V-A: the 28-layer backbone is decoded with temperature 0.7 and top_p 0.9;
 * the 40-layer one greedily).  After this call every decode step draws each sequence's token from
 * the nucleus of its exit head's logits instead of taking their arg max: over the ids of the step's
 * modality, p = softmax(z / temperature); ids in decreasing p (equal p: lower id first); the
 * shortest prefix whose mass reaches top_p is kept; the token is the first id whose cumulative
 * mass exceeds u * (kept mass).  u comes from `uniforms` (DEVICE float [max_seqs], borrowed until
 * the next call of this function): the step reads uniforms[i] in [0, 1) for the i-th sequence of
 * its `slots` argument, so the caller refills the array before each step on the same stream; no
 * random numbers are generated inside the library.  `scratch` (DEVICE, 16-byte aligned, at least
 * sparsk_sampling_scratch_bytes(dims), borrowed) holds the logits of a step.  Exit depths, the
 * pending sets and the cache are unaffected by how the token is chosen.
 * uniforms == NULL switches back to greedy decoding.  SPARSK_EINVAL for temperature <= 0 or not
 * finite, top_p outside (0, 1], a missing, misaligned or short scratch; SPARSK_ECAPACITY if a
 * modality has more than 196,608 ids (what one cluster of the sampling kernel holds in registers). */
size_t sparsk_sampling_scratch_bytes(const sparsk_dims *dims /*host*/);
int sparsk_set_sampling(sparsk_ctx *ctx, float temperature, float top_p, const float *uniforms /*device*/,
                        void *scratch /*device*/, size_t scratch_bytes);

/* The sampling kernel on its own: row i of `logits` (DEVICE float [n][vocab_text + vocab_speech])
 * is sampled over ids [0, vocab_text) if modality[i] == 0, else over [vocab_text, vocab_text +
 * vocab_speech), with uniforms[i]; tokens[i] receives the id (-1 if the range is empty).  All
 * array arguments are DEVICE pointers; nothing else is written.  Enqueued on `cuda_stream`;
 * SPARSK_EINVAL for NULL pointers, n < 1, vocab_text < 1, vocab_speech < 0, a range of more than
 * 196,608 ids, temperature <= 0 or top_p outside (0, 1]. */
int sparsk_nucleus_sample(const float *logits, const float *uniforms, const int32_t *modality, int32_t n,
                          int32_t vocab_text, int32_t vocab_speech, float temperature, float top_p,
                          int32_t *tokens, void *cuda_stream);

/* Stand-alone split-KV grouped-query attention: the two kernels a decode step runs per layer
 * (partials per KV split, then the merge), on caller-described rows.  Rows are grouped: group g
 * is rows [grp_row0[g], grp_row0[g] + grp_nrows[g]) of ONE sequence at consecutive positions;
 * the groups must partition [0, n_rows) (every row in exactly one group) and no group may have
 * more than max_grp_rows rows: a row outside every group, or beyond an under-stated
 * max_grp_rows, gets whatever the scratch held;
 * row i of a group attends to cache positions 0..row_pos[i] of slot row_slot[i] (the causal
 * block of Algorithm 1's full-depth branch on top of the earlier cache; a lower-pass row is a
 * group of one).  All array pointers are DEVICE pointers.  Rows whose slot is outside
 * [0, n_slots) or whose position is outside the cache read nothing and produce zeros.
 * `scratch` (device, 256-byte aligned, >= sparsk_attention_scratch_bytes) is overwritten. */
typedef struct {
    const void *q;               /* bf16 [n_rows][n_q_heads*head_dim], rotated queries             */
    const void *k_cache;         /* fp16 [n_slots][n_kv_heads][cache_len][head_dim], rotated keys  */
    const void *v_cache;         /* fp16, same layout                                              */
    void *out;                   /* bf16 [n_rows][n_q_heads*head_dim]                              */
    const int32_t *row_slot, *row_pos;     /* [n_rows]                                             */
    const int32_t *grp_row0, *grp_nrows;   /* [n_groups]                                           */
    int32_t n_rows, n_groups;
    int32_t max_grp_rows;        /* host-known bound on grp_nrows                                  */
    int32_t max_len;             /* host-known bound on row_pos + 1                                */
    int32_t n_q_heads, n_kv_heads, head_dim /* 64 or 128 */, cache_len, n_slots;
} sparsk_attn_args;
/* Bytes of scratch sparsk_attention needs (no counterpart in the paper: memory management). */
size_t sparsk_attention_scratch_bytes(int32_t n_rows, int32_t n_q_heads, int32_t head_dim);
int sparsk_attention(const sparsk_attn_args *args /*host*/, void *scratch /*device*/, size_t scratch_bytes,
                     void *cuda_stream);

/* The same attention for callers that cannot allocate device memory (no counterpart in the
 * paper: this exists for integration only).  Typical callers: a plug-in inside another engine
 * whose memory plan leaves no allocator to call, code on a path where cudaMalloc is forbidden
 * because it synchronises the device, a process whose device pool belongs to another runtime.
 * The split partials go to a fixed area of SPARSK_STATIC_SCRATCH_BYTES that is part of the
 * library image; every GPU that loads the library holds it until the process exits.  The call
 * allocates nothing and frees nothing.
 *   - A call whose partials do not fit (sparsk_attention_scratch_bytes(n_rows, n_q_heads,
 *     head_dim) > SPARSK_STATIC_SCRATCH_BYTES) is refused with SPARSK_ECAPACITY before anything
 *     is launched; `err` (host buffer, may be NULL) then says how much was needed.
 *   - The first call on each device looks up the area's device address (with that device
 *     current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one area, which keeps the previous call's contents;
 *     nothing in it needs clearing between calls.  Two calls that overlap on the GPU (different
 *     streams, no ordering between them) race on it: order them.
 * Arguments, layouts and results are those of sparsk_attention. */
#define SPARSK_STATIC_SCRATCH_BYTES (8u << 20)
int sparsk_attention_static(const sparsk_attn_args *args /*host*/, void *cuda_stream, char *err /*host*/,
                            size_t err_len);

/* Per-kernel timing for roofline reports.  sparsk_set_option(ctx, "time_kernel", c) with c =
 * 1 QKV, 2 attention, 3 O-projection, 4 gate/up, 5 down-projection, 6 exit head, 7 persistent layer-range kernel (8: all of them, see sparsk_kernel_time_by_class) brackets every
 * later launch of that class with CUDA events on the context's stream (up to 16384 launches; 0
 * stops).  sparsk_kernel_time synchronises the stream and returns the summed device time of the
 * bracketed launches and their number.  No counterpart in the paper: measurement only. */
int sparsk_kernel_time(sparsk_ctx *ctx, double *total_ms /*host*/, int64_t *n_launches /*host*/);
/* No counterpart in the paper (measurement only).  With "time_kernel" = 8 every launch is
 * bracketed and remembered with its class; this returns
 * the summed device time and the launch count of each class, indexed 0 bookkeeping (schedule,
 * compaction, embedding, norms, stash, gather, finish), 1..7 as above.  Arrays of 8. */
int sparsk_kernel_time_by_class(sparsk_ctx *ctx, double *total_ms /*host [8]*/, int64_t *n_launches /*host [8]*/);

/* Synchronises the context's stream, then reads and clears the device status word that kernels
 * raise instead of trapping: SPARSK_ETIMEOUT if a bounded in-kernel wait ran out, SPARSK_EINVAL
 * if a token id had to be clamped into the vocabulary, else SPARSK_OK.  After SPARSK_ETIMEOUT
 * the kernels' barrier state has been reset; the slots of the step that timed out hold an
 * incomplete step and must be reset before further use.  No counterpart in the paper: error
 * reporting only. */
int sparsk_check(sparsk_ctx *ctx);

/* Phase clock of the persistent layer-range kernel: its first CTA records the GPU's nanosecond
 * timer when it starts and after each of the six phases of every layer (q/k/v, attention,
 * merge, O-projection, gate/up, down-projection).  Copies the entries of the most recent launch
 * to out_ns (host), synchronising the stream; returns how many were written (at most
 * `capacity`), or a negative code.  No counterpart in the paper: measurement only. */
int sparsk_phase_trace(sparsk_ctx *ctx, int64_t *out_ns /*host*/, int32_t capacity);

/* Number of kernels this library has launched on behalf of the context so far.  No counterpart
 * in the paper: measurement only. */
int64_t sparsk_launch_count(const sparsk_ctx *ctx);

/* Confidence-based exit (Sec. V-B): the entropies the last decode step saw.  out[i * L + l] is
 * the entropy of head g_l's prediction for the i-th sequence of that step (l in [conf_start, L)),
 * or -1 where the head was not consulted (the sequence had left, or follows the schedule).  Host
 * array of n_seqs * L floats; n_seqs at most the last step's.  Parity hook: a checker can judge
 * the depths the step chose against entropies of its own. */
int sparsk_conf_entropies(const sparsk_ctx *ctx, int32_t n_seqs, float *out /*host*/);

/* Which implementation the layer passes so far went through (a pass = one layer over one row
 * set): layer_passes[0] persistent layer-range kernel (1-2 rows), [1] tcgen05 kernels launched
 * per projection, [2] small-batch GEMV kernels.  Lets a benchmark
 * attribute bytes to the kernel it times without re-deriving the choice.  No counterpart in the
 * paper: measurement only. */
int sparsk_route_counts(const sparsk_ctx *ctx, int64_t *layer_passes /*host [3]*/);

/* Text of the last error of this context (host string, valid until the next call).  No
 * counterpart in the paper: error reporting only. */
const char *sparsk_last_error(const sparsk_ctx *ctx);

/* Release host-side state.  The workspace and weights are the caller's to free.  The pointer
 * is dead afterwards: passing it to any call is undefined (SPARSK_ESTATE is returned only for
 * NULL and for memory that is recognisably not a live context).  No counterpart in the paper. */
int sparsk_destroy(sparsk_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* SPARSK_H */

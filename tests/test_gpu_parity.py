"""GPU parity: the CUDA library through its C ABI against the C oracle, element by element."""
import numpy as np
import pytest
import torch

from paper_2603_09215_b200 import synth

pytestmark = pytest.mark.gpu

MICRO64 = dict(n_layers=3, d_model=136, n_q_heads=6, n_kv_heads=2, head_dim=64, d_ffn=200,
               vocab_text=301, vocab_speech=99, rms_eps=1e-6, rope_base=10000.0)


@pytest.fixture(scope="module")
def util():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity_util
    return parity_util


def test_config1_tiny_full_run(util):
    """Workload 1 in full: 32-token prompt, 96 steps, 2 text : 4 speech, e=2, K=3."""
    wl = synth.WORKLOADS["cfg1_tiny_b1"]
    dims = synth.model_dims("tiny", wl["exit_layer"], wl["refresh_period"], wl["refresh_phase"])
    w = synth.make_weights(dims, seed=0)
    prompt = synth.make_prompts(dims, 1, 32, 32)[0]
    P = util.Pair(dims, w, 1, 32 + 96 + 1, wl["refresh_period"] - 1)
    P.prefill([prompt])
    P.check_cache(0, range(1, 5), 31)
    depths = []
    for g in range(wl["steps"]):
        m, c = synth.interleave(g, wl["n_text"], wl["n_speech"])
        ref, _, dep = P.step([m], [c])
        depths.append(int(dep[0]))
        if ref[0]["depth"] == 4:       # after a full-depth step the whole cache is complete
            P.check_cache(0, range(1, 5), 32 + g)
    sp = [d for g, d in enumerate(depths) if synth.interleave(g, 2, 4)[0] == 1]
    assert sp[:4] == [4, 2, 2, 4] and sum(sp) / len(sp) == 3.0
    assert P.stats["tok_checked"] > 40, P.stats
    print("cfg1", P.stats)
    P.close()


@pytest.mark.parametrize("min_rows", [3, 1])
@pytest.mark.parametrize("e,K,r,nt,ns", [(1, 2, 0, 1, 4), (2, 4, 1, 2, 7), (3, 2, 0, 1, 4), (2, 1, 0, 1, 4),
                                          (1, 5, 4, 0, 9)])
def test_odd_shapes_and_schedules(util, e, K, r, nt, ns, min_rows):
    """head_dim 64, 3 query heads per kv head, dimensions that are not multiples of the 256-wide
    chunks, vocabulary ranges that are not multiples of the row groups; several (e, K, r)."""
    dims = synth.model_dims(MICRO64, e, K, r)
    w = synth.make_weights(dims, seed=5)
    prompt = synth.make_prompts(dims, 1, 37, 37, seed=7)[0]
    P = util.Pair(dims, w, 1, 128, 2 * K, prefill_rows=16, options={"gemm_min_rows": min_rows})
    P.prefill([prompt])
    for g in range(40):
        m, c = synth.interleave(g, nt, ns)
        P.step([m], [c])
    P.check_cache(0, range(1, 4), P.g.slot_state(0)[0] - P.g.slot_state(0)[1])
    P.close()


@pytest.mark.parametrize("min_rows,trim", [(3, 1), (1, 2), (1 << 30, 2), (3, 0), (3, 2)])
def test_heterogeneous_batch_matches_per_sequence_oracle(util, min_rows, trim):
    """Batch of 7 with random interleave phases and counter offsets and ragged prompts, so every
    step mixes text, early-exit and refresh rows; sequences stay independent.  Run with the
    default hand-over between the small-batch and the tensor-core path (3 rows), with every
    projection on the tensor cores, and with every projection on the small-batch path; and with the pending rows leaving
    the last layer after its K/V projection (trim 2: always, 1: when it pays, 0: never), which
    must change nothing: the cache of every layer is compared below."""
    dims = synth.model_dims("tiny", 2, 4, 0)
    w = synth.make_weights(dims, seed=0)
    B = 7
    prompts = synth.make_prompts(dims, B, 9, 70, seed=4)
    phi, off = synth.make_phases(B, 1, 4, 4, True, seed=8)
    P = util.Pair(dims, w, B, 70 + 64, 3, prefill_rows=24, options={"gemm_min_rows": min_rows, "trim_last_layer": trim})
    P.prefill(prompts)
    mixed = 0
    for g in range(48):
        mc = [synth.interleave(g, 1, 4, int(p), int(o)) for p, o in zip(phi, off)]
        ref, _, dep = P.step([m for m, _ in mc], [c for _, c in mc])
        mixed += len(set(int(x) for x in dep)) > 1
    assert mixed > 20
    for s in range(B):
        ln, pend = P.g.slot_state(s)
        P.check_cache(s, range(1, 3), ln)          # lower layers are always complete
        P.check_cache(s, range(3, 5), ln - pend)   # upper layers up to the last full step
    print("hetero", P.stats)
    P.close()


MICRO128 = dict(n_layers=3, d_model=192, n_q_heads=8, n_kv_heads=1, head_dim=128, d_ffn=320,
                vocab_text=211, vocab_speech=77, rms_eps=1e-6, rope_base=10000.0)


@pytest.mark.parametrize("min_q,split", [(33, 0), (1, 0), (1, 64)])
def test_tensor_core_attention_for_blocks_of_query_vectors(util, min_q, split):
    """head_dim 128 with eight query heads per kv head: flushes of five pending rows + current
    (48 query vectors), prefill chunks of 24 rows (192 query vectors = two blocks of 128) and,
    with min_q = 1, single rows too go through the tcgen05 attention kernel; with 64-position
    splits a pass has several KV splits and ragged last tiles."""
    dims = synth.model_dims(MICRO128, 1, 6, 0)
    w = synth.make_weights(dims, seed=3)
    B = 3
    prompts = synth.make_prompts(dims, B, 70, 150, seed=12)
    P = util.Pair(dims, w, B, 150 + 64, 5, prefill_rows=24,
                  options={"attn_tc_min_q": min_q, "attn_split": split})
    P.prefill(prompts)
    for s in range(B):
        P.check_cache(s, range(1, 4), len(prompts[s]) - 1)
    phases = [0, 3, 5]
    for g in range(30):
        mc = [synth.interleave(g, 1, 6, ph) for ph in phases]
        P.step([m for m, _ in mc], [c for _, c in mc])
    for s in range(B):
        ln, pend = P.g.slot_state(s)
        P.check_cache(s, range(1, 2), ln)
        P.check_cache(s, range(2, 4), ln - pend)
    print("tc attention", P.stats)
    P.close()


def test_subset_of_slots_and_slot_reuse(util):
    """Steps may name any subset of slots in any order; a reset slot starts over."""
    dims = synth.model_dims("tiny", 2, 3, 0)
    w = synth.make_weights(dims, seed=0)
    prompts = synth.make_prompts(dims, 3, 12, 20, seed=2)
    P = util.Pair(dims, w, 3, 96, 2)
    P.prefill(prompts)
    for g in range(6):
        P.step([1, 1, 1], [g % 4] * 3)
    for g in range(6):
        P.step([1, 0], [g % 4, 0], slots=[2, 0])
    P.step([0], [0], slots=[1])
    # reuse slot 1 for a new sequence
    P.g.reset_slot(1)
    P.os[1] = P.om.new_seq(2)
    newp = synth.make_prompts(dims, 1, 15, 15, seed=9)[0]
    P.g.prefill([1], [newp[:-1]])
    P.os[1].prefill(newp[:-1])
    P.next_in[1] = int(newp[-1])
    for g in range(8):
        P.step([1, 1, 1], [g % 4] * 3, slots=[1, 2, 0])
    P.close()


def test_imported_cache_long_context(util):
    """A long synthetic cache (several KV splits and tiles, ragged tail) loaded into both sides."""
    dims = synth.model_dims("tiny", 2, 4, 0)
    w = synth.make_weights(dims, seed=0)
    n = 1000 + 37
    k, v = synth.synth_kv(dims, n, seed=6)
    P = util.Pair(dims, w, 2, n + 40, 3)
    from oracle.bruteforce import bf16_to_f64
    for layer in range(1, 5):
        kt = torch.from_numpy(k[layer - 1].view(np.int16)).cuda().view(torch.bfloat16).to(torch.float16)
        vt = torch.from_numpy(v[layer - 1].view(np.int16)).cuda().view(torch.bfloat16).to(torch.float16)
        for s in range(2):
            P.g.import_kv(s, layer, 0, kt, vt)
        kf, vf = bf16_to_f64(k[layer - 1]), bf16_to_f64(v[layer - 1])
        for s in range(2):
            for p in range(n):
                P.os[s].set_kv(layer, p, kf[p], vf[p])
    for s in range(2):
        P.g.set_len(s, n)
        P.os[s].set_len(n)
    P.next_in = [3, 1030]
    for g in range(12):
        mc = [synth.interleave(g, 1, 4, ph, 0) for ph in (0, 2)]
        P.step([m for m, _ in mc], [c for _, c in mc])
    print("long", P.stats)
    P.close()


def test_host_step_and_error_codes(util):
    from paper_2603_09215_b200 import binding
    dims = synth.model_dims("tiny", 2, 3, 0)
    w = synth.make_weights(dims, seed=0, head_layers=[2, 4])
    P = util.Pair(dims, w, 2, 40, 1)
    prompts = synth.make_prompts(dims, 2, 10, 10, seed=3)
    P.prefill(prompts)
    nt, dp = np.zeros(2, np.int32), np.zeros(2, np.int32)
    ref = [P.os[s].decode_step(P.next_in[s], 1, 0) for s in range(2)]
    P.g.decode_step_host([0, 1], P.next_in, [1, 1], [0, 0], nt, dp)
    assert list(dp) == [4, 4]
    for s in range(2):
        if ref[s]["margin"] > util.MARGIN:
            assert nt[s] == ref[s]["token"]
    before = [P.g.slot_state(s) for s in range(2)]
    with pytest.raises(binding.SparskError) as ei:      # repeated slot
        P.g.decode_step_host([0, 0], [1, 1], [1, 1], [1, 1], nt, dp)
    assert ei.value.code == binding.EINVAL
    P.g.decode_step_host([0, 1], [5, 6], [1, 1], [1, 1], nt, dp)           # early exit: 1 pending
    assert list(dp) == [2, 2]
    with pytest.raises(binding.SparskError) as ei:      # a second pending position does not fit
        P.g.decode_step_host([0, 1], [5, 6], [1, 1], [2, 2], nt, dp)
    assert ei.value.code == binding.ECAPACITY
    assert [P.g.slot_state(s) for s in range(2)] == [(b[0] + 1, 1) for b in before]
    before = [P.g.slot_state(s) for s in range(2)]
    with pytest.raises(binding.SparskError) as ei:      # token outside the vocabulary: refused on the host
        P.g.decode_step_host([0], [10 ** 6], [0], [0], nt, dp)
    assert ei.value.code == binding.EINVAL
    assert [P.g.slot_state(s) for s in range(2)] == before      # nothing ran, nothing advanced
    P.g.check()
    P.close()
    # a schedule that needs a head that was not supplied
    d2 = synth.model_dims("tiny", 3, 3, 0)
    gw = binding.upload_weights(w)
    with pytest.raises(binding.SparskError) as ei:
        binding.Sparsk(d2, gw, 1, 16, 2)
    assert ei.value.code == binding.ENOHEAD


@pytest.mark.parametrize("options", [{"mega": 0}, {"mega_max_rows": 4}, {"mega_max_rows": 1, "gemm_min_rows": 2},
                                     {"mega": 0, "gemm_min_rows": 1 << 30}, {"gemm_kb": 1, "mega": 0, "gemm_min_rows": 1},
                                     {"trim_last_layer": 2}, {"trim_last_layer": 2, "mega": 0, "gemm_min_rows": 1},
                                     {"trim_last_layer": 2, "mega": 0, "gemm_min_rows": 1 << 30}, {"trim_last_layer": 0}])
def test_every_route_for_small_passes(util, options):
    """Passes of 1..4 rows (K = 4: flushes of up to three pending rows) through each of the
    implementations: the persistent kernel (also with its moving activation window at 3-4 rows),
    the tensor-core path (with 2-D descriptors too) and the small-batch kernels."""
    dims = synth.model_dims("tiny", 2, 4, 0)
    w = synth.make_weights(dims, seed=0)
    prompt = synth.make_prompts(dims, 1, 21, 21, seed=11)[0]
    P = util.Pair(dims, w, 1, 96, 3, prefill_rows=16, options=options)
    P.prefill([prompt])
    for g in range(25):
        m, c = synth.interleave(g, 1, 4)
        P.step([m], [c])
    ln, pend = P.g.slot_state(0)
    P.check_cache(0, range(1, 5), ln - pend)
    P.close()


@pytest.mark.parametrize("options", [{"attn_ctas": 2, "attn_split": 16, "mega": 0}, {"attn_ctas": 2, "attn_split": 32, "mega": 0},
                                     {"attn_ctas": 3, "attn_split": 48, "mega": 0, "attn_stages": 3},
                                     {"attn_ctas": 1, "attn_split": 64, "mega": 0, "attn_tma": 0},
                                     {"attn_ctas": 2, "attn_split": 16, "mega": 0, "attn_dynamic": 0},
                                     {"attn_ctas": 1, "mega": 0, "gemm_min_rows": 1}])
def test_attention_items_drawn_from_the_counter(util, options):
    """Many more attention work items than warps (the kernel held to one or two CTAs, four ragged
    sequences, short splits): the warps draw items from the ticket counter, launch after launch
    (the host predicts the counter's value instead of resetting it), or take every n-th item.
    Splits of one, two and three tiles with ragged ends, so that items shorter than, as long as and
    longer than a warp's ring follow one another and each starts its successor's first tiles."""
    dims = synth.model_dims("tiny", 2, 4, 0)
    w = synth.make_weights(dims, seed=0)
    prompts = synth.make_prompts(dims, 4, 9, 150, seed=21)
    P = util.Pair(dims, w, 4, 200, 3, prefill_rows=16, options=options)
    P.prefill(prompts)
    for g in range(14):
        mc = [synth.interleave(g + 2 * i, 1, 4) for i in range(4)]
        P.step([m for m, _ in mc], [c for _, c in mc])
    for s_ in range(4):
        ln, pend = P.g.slot_state(s_)
        P.check_cache(s_, range(1, 5), ln - pend)
    P.close()


def test_timeout_is_reported_once_and_the_context_recovers(util):
    """A bounded in-kernel wait that runs out: the persistent kernel is told a grid-barrier count
    that no CTA can reach (a host-side test hook; nothing faults or hangs), its wait ends at the
    wall-clock limit, every CTA leaves, and the step returns SPARSK_ETIMEOUT exactly once.  The
    library then resets its barrier state by itself: after the caller resets the slot that took
    part, decoding matches the oracle again."""
    from paper_2603_09215_b200 import binding
    dims = synth.model_dims("tiny", 2, 3, 0)
    w = synth.make_weights(dims, seed=0)
    prompt = synth.make_prompts(dims, 1, 14, 14, seed=5)[0]
    P = util.Pair(dims, w, 1, 64, 2)
    P.prefill([prompt])
    for g in range(4):
        m, c = synth.interleave(g, 2, 4)
        P.step([m], [c])
    assert P.g.route_counts()["mega"] > 0                 # the steps above ran in the persistent kernel
    nt, dp = np.zeros(1, np.int32), np.zeros(1, np.int32)
    P.g.set_option("inject_barrier_timeout", 1)
    with pytest.raises(binding.SparskError) as ei:
        P.g.decode_step_host([0], [P.next_in[0]], [1], [0], nt, dp)
    assert ei.value.code == binding.ETIMEOUT
    P.g.check()                                           # reported once; the status word is clear again
    # the interrupted step left slot 0 incomplete: start it over on both sides
    P.g.reset_slot(0)
    P.os[0] = P.om.new_seq(2)
    P.g.prefill([0], [prompt[:-1]])
    P.os[0].prefill(prompt[:-1])
    P.next_in[0] = int(prompt[-1])
    for g in range(12):
        m, c = synth.interleave(g, 2, 4)
        P.step([m], [c])
    ln, pend = P.g.slot_state(0)
    P.check_cache(0, range(1, 5), ln - pend)
    P.close()


MICRO256 = dict(n_layers=3, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=512,
                vocab_text=301, vocab_speech=99, rms_eps=1e-6, rope_base=10000.0)


@pytest.mark.parametrize("K,maxp", [(4, 3), (3, 2)])
def test_persistent_kernel_tensor_core_form_for_three_and_four_rows(util, K, maxp):
    """Flushes of two and three pending rows (passes of three and four rows) inside the persistent
    layer-range kernel: its tensor-core form (swizzled weight boxes, mma.sync, two-term
    activations), on a shape whose inner dimensions are whole 64-element blocks."""
    dims = synth.model_dims(MICRO256, 1, K, 0)
    w = synth.make_weights(dims, seed=9)
    prompt = synth.make_prompts(dims, 1, 23, 23, seed=2)[0]
    P = util.Pair(dims, w, 1, 23 + 64, maxp, prefill_rows=16, options={"mega_max_rows": 4})
    P.prefill([prompt])
    before = P.g.route_counts()
    for g in range(30):
        m, c = synth.interleave(g, 1, K)
        P.step([m], [c])
    after = P.g.route_counts()
    assert after["tc"] == before["tc"] and after["gemv"] == before["gemv"]      # every decode pass ran in the persistent kernel
    assert P.stats["max_flush"] == K - 1
    ln, pend = P.g.slot_state(0)
    P.check_cache(0, range(1, 4), ln - pend)
    print("mega tc", P.stats)
    P.close()

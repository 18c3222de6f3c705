"""Pins for the C oracle's decoder: cache-free recomputation, a library Llama forward,
textbook identities of its sub-blocks, and the KV invariant of Sec. IV-B.3."""
import numpy as np
import pytest

from oracle import bruteforce as bf
from oracle import oracle as ora
from paper_2603_09215_b200 import synth

MICRO = dict(n_layers=3, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ffn=48,
             vocab_text=40, vocab_speech=24, rms_eps=1e-6, rope_base=10000.0)


def _run_oracle(dims, w, prompt, mods, ctrs, max_pending=16, forced=None):
    m = ora.OracleModel(dims, w, max_len=len(prompt) + len(mods) + 1)
    s = m.new_seq(max_pending)
    s.prefill(prompt[:-1])
    tok = int(prompt[-1])
    out = []
    for i, (mod, c) in enumerate(zip(mods, ctrs)):
        r = s.decode_step(tok, mod, c)
        r["pending_after"] = s.pending
        out.append(r)
        tok = int(forced[i]) if forced is not None else r["token"]
    return m, s, out


def _sched(steps, n_text, n_speech, phase=0, offset=0):
    mc = [synth.interleave(g, n_text, n_speech, phase, offset) for g in range(steps)]
    return [m for m, _ in mc], [c for _, c in mc]


@pytest.mark.parametrize("e,K,r,nt,ns,phase", [
    (1, 2, 0, 1, 4, 0), (2, 3, 0, 2, 4, 0), (2, 2, 1, 1, 5, 2), (1, 4, 2, 2, 7, 1),
    (3, 3, 0, 1, 4, 0), (2, 1, 0, 1, 4, 0), (2, 5, 4, 0, 9, 0)])
def test_matches_cache_free_recomputation(e, K, r, nt, ns, phase):
    dims = synth.model_dims(MICRO, e, K, r)
    w = synth.make_weights(dims, seed=11)
    prompt = synth.make_prompts(dims, 1, 5, 5, seed=5)[0]
    mods, ctrs = _sched(22, nt, ns, phase)
    _, _, got = _run_oracle(dims, w, prompt, mods, ctrs)
    ref = bf.decode_stream(dims, w, prompt, mods, ctrs)
    assert [g["depth"] for g in got] == [x["depth"] for x in ref]
    assert [g["token"] for g in got] == [x["token"] for x in ref]
    Vt, V = dims["vocab_text"], dims["vocab_text"] + dims["vocab_speech"]
    for g, x, mod in zip(got, ref, mods):
        np.testing.assert_allclose(g["hidden"], x["hidden"], rtol=1e-9, atol=1e-11)
        lo, hi = (0, Vt) if mod == 0 else (Vt, V)
        np.testing.assert_allclose(g["logits"][lo:hi], x["logits"][lo:hi], rtol=1e-9, atol=1e-11)
        assert np.isneginf(np.delete(g["logits"], np.s_[lo:hi])).all()
        assert abs(g["margin"] - x["margin"]) < 1e-9


@pytest.mark.parametrize("text_exit,K,r,nt,ns,running,tp,tr", [
    (1, 2, 0, 3, 4, False, 0, 0),    # text and speech both follow Even
    (2, 2, 0, 5, 3, False, 0, 0),    # text only (Sec. V-E row G10); speech flushes the pending text rows
    (0, 6, 5, 1, 5, False, 0, 0),    # fixed-layer exit: no refresh inside a chunk, the text step flushes 5 rows
    (0, 3, 0, 1, 4, True, 0, 0),     # counter running across chunks instead of restarting
    (0, 2, 1, 1, 4, False, 0, 0),    # Odd
    (1, 4, 0, 6, 8, False, 3, 1),    # a period and phase of its own for each modality (Sec. V-E)
    (2, 2, 0, 6, 2, False, 3, 2)])   # text only, with its own period
def test_schedule_variants_match_cache_free_recomputation(text_exit, K, r, nt, ns, running, tp, tr):
    """The schedule variants of Sec. IV-B.1 / V-B / V-E: whatever the caller's counters make of the
    depths, pending rows persist until the next full-depth step of either modality and the stream
    equals cache-free recomputation."""
    dims = synth.model_dims(MICRO, 2, K, r, text_exit=text_exit, text_period=tp, text_phase=tr)
    w = synth.make_weights(dims, seed=13)
    prompt = synth.make_prompts(dims, 1, 6, 6, seed=3)[0]
    mc = [synth.interleave(g, nt, ns, running=running) for g in range(26)]
    mods, ctrs = [m for m, _ in mc], [c for _, c in mc]
    _, _, got = _run_oracle(dims, w, prompt, mods, ctrs)
    ref = bf.decode_stream(dims, w, prompt, mods, ctrs)
    assert [g["depth"] for g in got] == [x["depth"] for x in ref]
    assert [g["token"] for g in got] == [x["token"] for x in ref]
    for g, x in zip(got, ref):
        np.testing.assert_allclose(g["hidden"], x["hidden"], rtol=1e-9, atol=1e-11)
    depths = [g["depth"] for g in got]
    assert 2 in depths and 3 in depths
    if text_exit == 2:
        assert all(d == 3 for d, m in zip(depths, mods) if m == 1)
        assert any(d == 2 for d, m in zip(depths, mods) if m == 0)
    if tp:       # each modality follows its own (period, phase): text counters are in-chunk indices
        assert [d for d, m in zip(depths, mods) if m == 0] == [3 if c % tp == tr else 2 for c, m in zip(ctrs, mods) if m == 0]
        if text_exit == 1:
            assert [d for d, m in zip(depths, mods) if m == 1] == [3 if c % K == r else 2 for c, m in zip(ctrs, mods) if m == 1]
    if K == 6:   # fixed-layer: every speech step leaves early, pending reaches the chunk length
        assert all(d == 2 for d, m in zip(depths, mods) if m == 1)
        assert max(len(g["pending_after"]) for g in got) == ns


def test_config1_full_run_matches_cache_free_recomputation():
    wl = synth.WORKLOADS["cfg1_tiny_b1"]
    dims = synth.model_dims("tiny", wl["exit_layer"], wl["refresh_period"], wl["refresh_phase"])
    w = synth.make_weights(dims, seed=0)
    prompt = synth.make_prompts(dims, 1, 32, 32)[0]
    mods, ctrs = _sched(wl["steps"], wl["n_text"], wl["n_speech"])
    _, _, got = _run_oracle(dims, w, prompt, mods, ctrs)
    ref = bf.decode_stream(dims, w, prompt, mods, ctrs, forced=[g["token"] for g in got])
    assert [g["depth"] for g in got] == [x["depth"] for x in ref]
    for g, x in zip(got, ref):
        np.testing.assert_allclose(g["hidden"], x["hidden"], rtol=1e-8, atol=1e-10)
        if x["margin"] > 1e-9:
            assert g["token"] == x["token"]
    sp = [g["depth"] for g, m in zip(got, mods) if m == 1]
    assert sum(sp) / len(sp) == 3.0


def test_kv_invariant_and_pending_set():
    """After every full-depth step K/V at all layers equals the plain causal forward for all
    positions; between them, upper layers are filled exactly up to the last full step and the
    pending set is the run of early-exit positions since then (at most K-1 of them)."""
    e, K = 1, 3
    dims = synth.model_dims(MICRO, e, K, 0)
    w = synth.make_weights(dims, seed=3)
    prompt = synth.make_prompts(dims, 1, 4, 4, seed=9)[0]
    mods, ctrs = _sched(20, 1, 7)
    m = ora.OracleModel(dims, w, max_len=64)
    s = m.new_seq(8)
    s.prefill(prompt[:-1])
    toks = list(prompt)
    last_full = len(prompt) - 2
    saw_flush = 0
    for mod, c in zip(mods, ctrs):
        n_before = len(s.pending)
        r = s.decode_step(toks[-1], mod, c)
        p = len(toks) - 1
        fw = bf.forward_all(dims, w, toks)
        if r["depth"] == dims["n_layers"]:
            saw_flush = max(saw_flush, n_before + 1)
            last_full = p
            assert s.pending == []
        else:
            assert s.pending == list(range(last_full + 1, p + 1))
            assert len(s.pending) <= K - 1
        for layer in range(1, dims["n_layers"] + 1):
            upto = p if layer <= e else last_full
            for pos in range(upto + 1):
                k, v = s.get_kv(layer, pos)
                np.testing.assert_allclose(k, fw["K"][layer - 1, pos], rtol=1e-9, atol=1e-11)
                np.testing.assert_allclose(v, fw["V"][layer - 1, pos], rtol=1e-9, atol=1e-11)
            for pos in range(upto + 1, p + 1):   # deferred entries are still untouched
                k, v = s.get_kv(layer, pos)
                assert not k.any() and not v.any()
        toks.append(r["token"])
    assert saw_flush == K   # a flush of K-1 pending rows plus the current one happened


def test_early_exit_token_is_kept():
    """The full-depth pass over a pending position may disagree with the token emitted there;
    the emitted stream keeps the early-exit token."""
    dims = synth.model_dims(MICRO, 1, 2, 0)
    w = synth.make_weights(dims, seed=21)
    prompt = synth.make_prompts(dims, 1, 6, 6, seed=2)[0]
    mods, ctrs = _sched(30, 1, 4)
    _, _, got = _run_oracle(dims, w, prompt, mods, ctrs)
    toks = list(prompt) + [g["token"] for g in got]
    fw = bf.forward_all(dims, w, toks[:-1])
    Vt = dims["vocab_text"]
    disagree = 0
    for i, (g, mod) in enumerate(zip(got, mods)):
        p = len(prompt) - 1 + i
        z_e = bf.head_logits(dims, w, g["depth"], fw["H"][g["depth"], p])
        z_L = bf.head_logits(dims, w, dims["n_layers"], fw["H"][dims["n_layers"], p])
        lo, hi = (0, Vt) if mod == 0 else (Vt, Vt + dims["vocab_speech"])
        assert g["token"] == lo + int(np.argmax(z_e[lo:hi]))
        if g["depth"] < dims["n_layers"] and lo + int(np.argmax(z_L[lo:hi])) != g["token"]:
            disagree += 1
    assert disagree > 0


def test_period_one_and_last_layer_exit_are_plain_decoding():
    base = synth.model_dims(MICRO, 3, 1, 0)
    w = synth.make_weights(base, seed=4)
    prompt = synth.make_prompts(base, 1, 5, 5, seed=6)[0]
    mods, ctrs = _sched(16, 1, 4)
    _, _, a = _run_oracle(base, w, prompt, mods, ctrs)                               # e = L
    _, _, b = _run_oracle(synth.model_dims(MICRO, 1, 1, 0), w, prompt, mods, ctrs)   # K = 1
    _, _, c = _run_oracle(synth.model_dims(MICRO, 2, 3, 0), w, prompt, [0] * 16, list(range(16)))
    _, _, a0 = _run_oracle(base, w, prompt, [0] * 16, list(range(16)))
    assert all(x["depth"] == 3 for x in a + b + c)
    assert [x["token"] for x in a] == [x["token"] for x in b]
    assert [x["token"] for x in c] == [x["token"] for x in a0]                      # all text
    for x, y in zip(a, b):
        np.testing.assert_allclose(x["hidden"], y["hidden"], rtol=1e-10, atol=1e-12)


def _hf_model(dims, w):
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    V = dims["vocab_text"] + dims["vocab_speech"]
    kw = dict(vocab_size=V, hidden_size=dims["d_model"], intermediate_size=dims["d_ffn"],
              num_hidden_layers=dims["n_layers"], num_attention_heads=dims["n_q_heads"],
              num_key_value_heads=dims["n_kv_heads"], head_dim=dims["head_dim"],
              rms_norm_eps=dims["rms_eps"], attention_bias=False, mlp_bias=False,
              tie_word_embeddings=False, max_position_embeddings=512, hidden_act="silu")
    try:
        cfg = tr.LlamaConfig(rope_theta=dims["rope_base"], **kw)
    except TypeError:
        cfg = tr.LlamaConfig(rope_parameters={"rope_type": "default",
                                              "rope_theta": dims["rope_base"]}, **kw)
    cfg._attn_implementation = "eager"
    model = tr.LlamaForCausalLM(cfg).to(torch.float64).eval()
    t = lambda a: torch.from_numpy(bf.bf16_to_f64(a))
    sd = {"model.embed_tokens.weight": t(w["embed"]),
          "model.norm.weight": t(w["head_norm"][-1]), "lm_head.weight": t(w["head_proj"][-1])}
    for l in range(dims["n_layers"]):
        p = f"model.layers.{l}."
        sd[p + "input_layernorm.weight"] = t(w["attn_norm"][l])
        sd[p + "self_attn.q_proj.weight"] = t(w["wq"][l])
        sd[p + "self_attn.k_proj.weight"] = t(w["wk"][l])
        sd[p + "self_attn.v_proj.weight"] = t(w["wv"][l])
        sd[p + "self_attn.o_proj.weight"] = t(w["wo"][l])
        sd[p + "post_attention_layernorm.weight"] = t(w["mlp_norm"][l])
        sd[p + "mlp.gate_proj.weight"] = t(w["w_gate"][l])
        sd[p + "mlp.up_proj.weight"] = t(w["w_up"][l])
        sd[p + "mlp.down_proj.weight"] = t(w["w_down"][l])
    missing = model.load_state_dict(sd, strict=False)
    assert not [k for k in missing.missing_keys if "rotary" not in k], missing
    return model


def test_against_library_llama_forward():
    """Depth-L decoding equals a bias-free Llama-architecture causal forward from a library, and
    the intermediate h^(l) equal that library's per-layer hidden states."""
    import torch  # the library keeps its rotary table in float32, hence 5e-6 below
    dims = synth.model_dims(MICRO, 3, 1, 0)
    w = synth.make_weights(dims, seed=8)
    prompt = synth.make_prompts(dims, 1, 7, 7, seed=12)[0]
    mods, ctrs = _sched(10, 1, 4)
    _, _, got = _run_oracle(dims, w, prompt, mods, ctrs)
    toks = list(prompt) + [g["token"] for g in got][:-1]
    model = _hf_model(dims, w)
    with torch.no_grad():
        out = model(torch.tensor([toks]), output_hidden_states=True)
    logits = out.logits[0].numpy()
    for i, g in enumerate(got):
        p = len(prompt) - 1 + i
        fin = np.isfinite(g["logits"])
        np.testing.assert_allclose(g["logits"][fin], logits[p][fin], rtol=5e-6, atol=1e-7)
    # per-layer hidden states of the cache-free forward (and hence of the oracle, by the
    # recomputation test) against the library's; the library's last entry is post-norm.
    fw = bf.forward_all(dims, w, toks)
    for l in range(dims["n_layers"]):
        np.testing.assert_allclose(fw["H"][l], out.hidden_states[l][0].numpy(), rtol=5e-6,
                                   atol=1e-7)
    # an early-exit run's hidden state at depth e equals the library's layer-e state
    d2 = synth.model_dims(MICRO, 2, 2, 1)
    _, _, ee = _run_oracle(d2, w, prompt, mods, ctrs, forced=toks[len(prompt):] + [0])
    for i, g in enumerate(ee):
        if g["depth"] == 2:
            p = len(prompt) - 1 + i
            np.testing.assert_allclose(g["hidden"], out.hidden_states[2][0, p].numpy(),
                                       rtol=5e-6, atol=1e-7)


def test_sub_block_identities():
    rng = np.random.default_rng(0)
    one = np.full(16, 0x3F80, np.uint16)          # bf16 1.0
    x = rng.normal(size=16)
    y = ora.rmsnorm(x, one, 0.0)
    assert abs((y * y).mean() - 1.0) < 1e-12
    np.testing.assert_allclose(ora.rmsnorm(3.7 * x, one, 0.0), y, rtol=1e-12)
    two = np.full(16, 0x4000, np.uint16)          # bf16 2.0: the gain multiplies
    np.testing.assert_allclose(ora.rmsnorm(x, two, 0.0), 2 * y, rtol=1e-12)
    np.testing.assert_allclose(ora.rmsnorm(x, one, 0.5), x / np.sqrt((x * x).mean() + 0.5))
    # rope: identity at position 0, norm preserving, scores depend on p - u only
    q, k = rng.normal(size=8), rng.normal(size=8)
    np.testing.assert_array_equal(ora.rope(q, 0, 10000.0), q)
    assert abs(np.linalg.norm(ora.rope(q, 17, 10000.0)) - np.linalg.norm(q)) < 1e-12
    a = ora.rope(q, 9, 10000.0) @ ora.rope(k, 4, 10000.0)
    b = ora.rope(q, 25, 10000.0) @ ora.rope(k, 20, 10000.0)
    assert abs(a - b) < 1e-12
    # the first pair rotates by exactly pos radians: (1,0) -> (cos p, sin p) in slots (0, hd/2)
    e0 = np.zeros(8); e0[0] = 1.0
    r0 = ora.rope(e0, 3, 10000.0)
    assert abs(r0[0] - np.cos(3)) < 1e-12 and abs(r0[4] - np.sin(3)) < 1e-12
    # the last pair rotates by pos * base^(-(hd-2)/hd)
    e3 = np.zeros(8); e3[3] = 1.0
    r3 = ora.rope(e3, 5, 10000.0)
    th = 5 * 10000.0 ** (-6 / 8)
    assert abs(r3[3] - np.cos(th)) < 1e-12 and abs(r3[7] - np.sin(th)) < 1e-12
    # attention: weights sum to one, one key returns its value, uniform when keys are equal
    K, V = rng.normal(size=(5, 8)), rng.normal(size=(5, 8))
    out, wts = ora.attend(q, K, V)
    assert abs(wts.sum() - 1) < 1e-12
    s = K @ q / np.sqrt(8)
    ref = np.exp(s - s.max()); ref /= ref.sum()
    np.testing.assert_allclose(wts, ref, rtol=1e-12)
    np.testing.assert_allclose(out, ref @ V, rtol=1e-12)
    out1, _ = ora.attend(q, K[:1], V[:1])
    np.testing.assert_allclose(out1, V[0], rtol=1e-15)
    out2, w2 = ora.attend(q, np.tile(K[:1], (4, 1)), V[:4])
    np.testing.assert_allclose(w2, 0.25, rtol=1e-12)
    np.testing.assert_allclose(out2, V[:4].mean(0), rtol=1e-12)


def test_grouped_query_reduces_to_multi_head():
    """With the KV heads repeated so that H_kv = H_q the result is unchanged."""
    dims = synth.model_dims(MICRO, 2, 2, 0)
    w = synth.make_weights(dims, seed=14)
    prompt = synth.make_prompts(dims, 1, 5, 5, seed=3)[0]
    mods, ctrs = _sched(10, 1, 4)
    _, _, a = _run_oracle(dims, w, prompt, mods, ctrs)
    G, hd = dims["n_q_heads"] // dims["n_kv_heads"], dims["head_dim"]
    w2 = dict(w)
    rep = lambda m: np.repeat(m.reshape(dims["n_kv_heads"], hd, -1), G, axis=0).reshape(
        dims["n_q_heads"] * hd, -1).copy()
    w2["wk"] = [rep(m) for m in w["wk"]]
    w2["wv"] = [rep(m) for m in w["wv"]]
    dims2 = dict(dims, n_kv_heads=dims["n_q_heads"])
    _, _, b = _run_oracle(dims2, w2, prompt, mods, ctrs)
    assert [x["token"] for x in a] == [x["token"] for x in b]
    for x, y in zip(a, b):
        np.testing.assert_allclose(x["hidden"], y["hidden"], rtol=1e-10, atol=1e-12)


def test_imported_cache_equals_prefilled_cache():
    """Loading K/V through set_kv gives the same continuation as computing them."""
    dims = synth.model_dims(MICRO, 2, 2, 0)
    w = synth.make_weights(dims, seed=17)
    prompt = synth.make_prompts(dims, 1, 9, 9, seed=4)[0]
    mods, ctrs = _sched(8, 1, 4)
    m, s, a = _run_oracle(dims, w, prompt, mods, ctrs)
    s2 = m.new_seq(8)
    fw = bf.forward_all(dims, w, prompt[:-1])
    for layer in range(1, dims["n_layers"] + 1):
        for pos in range(len(prompt) - 1):
            s2.set_kv(layer, pos, fw["K"][layer - 1, pos], fw["V"][layer - 1, pos])
    s2.set_len(len(prompt) - 1)
    tok = int(prompt[-1])
    for mod, c, ref in zip(mods, ctrs, a):
        r = s2.decode_step(tok, mod, c)
        assert r["token"] == ref["token"]
        np.testing.assert_allclose(r["hidden"], ref["hidden"], rtol=1e-9, atol=1e-11)
        tok = r["token"]


def test_capacity_and_missing_head_errors():
    dims = synth.model_dims(MICRO, 1, 4, 0)
    w = synth.make_weights(dims, seed=1, head_layers=[3])
    m = ora.OracleModel(dims, w, max_len=8)
    s = m.new_seq(2)
    s.prefill(np.array([1, 2], np.int32))
    s.decode_step(3, 1, 0)                                  # full depth, head 3 present
    with pytest.raises(RuntimeError):
        s.decode_step(3, 1, 1)                              # needs head 1: missing

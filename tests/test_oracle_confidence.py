"""Pins for the oracle's exits at arbitrary layers and its confidence rule (Sec. V-B, compared
method 3; Sec. VI gives the thresholds 0.1 and 0.5).

What the paper and the mathematics fix: the entropy of a distribution (uniform: ln n; one
certain outcome: 0; a hand-worked two-point case; shift invariance); with a threshold of 0 no
position ever exits early, so decoding is plain full-depth decoding; with an infinite threshold
every position of the modality leaves at the start layer, i.e. fixed-layer exit; whatever the
depths, deferred filling makes every step equal to a cache-free causal forward (Sec. IV-B.3), so
the stream with exits at arbitrary, changing layers equals full recomputation; and with one exit
layer the general step is Algorithm 1 itself.  The averages the paper prints for its confidence
rows (S3, G3, G11) come from trained heads and cannot be reproduced here: parity unpinned."""
import numpy as np
import pytest

from oracle import bruteforce as bf
from oracle import oracle as ora
from paper_2603_09215_b200 import synth

MICRO = dict(n_layers=5, d_model=32, n_q_heads=4, n_kv_heads=2, head_dim=8, d_ffn=48,
             vocab_text=40, vocab_speech=24, rms_eps=1e-6, rope_base=10000.0)


def _run_dyn(dims, w, prompt, mods, ctrs, depths=None, max_pending=32):
    m = ora.OracleModel(dims, w, max_len=len(prompt) + len(mods) + 1)
    s = m.new_seq(max_pending)
    s.prefill(prompt[:-1])
    tok = int(prompt[-1])
    out = []
    for i, (mod, c) in enumerate(zip(mods, ctrs)):
        r = s.decode_step_dyn(tok, mod, c, 0 if depths is None else depths[i])
        r["pending_after"] = list(zip(s.pending, s.pending_fill))
        out.append(r)
        tok = r["token"]
    return m, s, out


def test_entropy_values():
    assert abs(ora.entropy(np.zeros(7)) - np.log(7)) < 1e-12                 # uniform
    assert abs(ora.entropy(np.full(151936, 3.25)) - np.log(151936)) < 1e-9   # uniform, shifted, large
    assert ora.entropy([0.0, 800.0, -5.0]) < 1e-12                            # one certain outcome
    # p = (1/4, 3/4): -(1/4 ln 1/4 + 3/4 ln 3/4), worked by hand = 0.562335...
    assert abs(ora.entropy([0.0, np.log(3.0)]) - 0.5623351446188083) < 1e-12
    assert abs(ora.entropy([1.0, 1.0]) - np.log(2)) < 1e-12
    z = np.array([0.3, -1.2, 2.0, 0.0, 0.7])
    assert abs(ora.entropy(z) - ora.entropy(z + 123.0)) < 1e-12              # shift invariance
    p = np.exp(z) / np.exp(z).sum()
    assert abs(ora.entropy(z) - float(-(p * np.log(p)).sum())) < 1e-12
    assert abs(bf.entropy(z) - float(-(p * np.log(p)).sum())) < 1e-12


def test_arbitrary_depths_equal_cache_free_recomputation():
    """Every step told to leave at its own layer (1..L, changing from step to step): positions are
    carried upwards by later steps exactly as far as those steps go, and every emitted token,
    hidden state and logit vector equals a cache-free causal forward of the sequence so far."""
    dims = synth.model_dims(MICRO, 2, 3, 0)
    w = synth.make_weights(dims, seed=21)
    prompt = synth.make_prompts(dims, 1, 7, 7, seed=4)[0]
    rng = np.random.Generator(np.random.PCG64(9))
    depths = [int(x) for x in rng.integers(1, 6, size=28)]
    depths[5] = 5
    depths[17] = 5
    mods = [int(x) for x in rng.integers(0, 2, size=28)]
    ctrs = list(range(28))
    _, s, got = _run_dyn(dims, w, prompt, mods, ctrs, depths)
    ref = bf.decode_stream(dims, w, prompt, mods, ctrs, depths=depths)
    assert [g["depth"] for g in got] == depths
    assert [g["token"] for g in got] == [x["token"] for x in ref]
    for g, x in zip(got, ref):
        np.testing.assert_allclose(g["hidden"], x["hidden"], rtol=1e-9, atol=1e-11)
        fin = np.isfinite(g["logits"])
        np.testing.assert_allclose(g["logits"][fin], x["logits"][fin], rtol=1e-9, atol=1e-11)
    # bookkeeping: a position's fill level is the deepest step since it left; a full-depth step empties the set
    for i, g in enumerate(got):
        if depths[i] == 5:
            assert g["pending_after"] == []
        else:
            assert all(f >= depths[i] for _, f in g["pending_after"])
            assert g["pending_after"][-1][1] == depths[i]
    # the cache is complete up to each position's fill level
    toks = list(prompt[:-1]) + [int(prompt[-1])] + [g["token"] for g in got[:-1]]
    fw = bf.forward_all(dims, w, toks)
    fill = {pos: f for pos, f in got[-1]["pending_after"]}
    for pos in range(len(toks)):
        for layer in range(1, fill.get(pos, 5) + 1):
            k, v = s.get_kv(layer, pos)
            np.testing.assert_allclose(k, fw["K"][layer - 1, pos], rtol=1e-9, atol=1e-11)
            np.testing.assert_allclose(v, fw["V"][layer - 1, pos], rtol=1e-9, atol=1e-11)


def test_single_exit_layer_is_algorithm_1():
    """With the schedule's depths the general step and the scheduled decoder are the same program."""
    dims = synth.model_dims(MICRO, 2, 3, 0)
    w = synth.make_weights(dims, seed=21)
    prompt = synth.make_prompts(dims, 1, 6, 6, seed=5)[0]
    mc = [synth.interleave(g, 2, 5) for g in range(24)]
    mods, ctrs = [m for m, _ in mc], [c for _, c in mc]
    _, _, dyn = _run_dyn(dims, w, prompt, mods, ctrs)           # no confidence modality: the schedule decides
    m = ora.OracleModel(dims, w, max_len=64)
    s = m.new_seq(8)
    s.prefill(prompt[:-1])
    tok = int(prompt[-1])
    for g, (mod, c) in zip(dyn, zip(mods, ctrs)):
        r = s.decode_step(tok, mod, c)
        assert (r["depth"], r["token"]) == (g["depth"], g["token"])
        np.testing.assert_array_equal(r["hidden"], g["hidden"])
        tok = r["token"]


def _conf_dims(thr, start=2, mods=2, **kw):
    return synth.model_dims(MICRO, 3, 2, 0, conf_modalities=mods, conf_start=start, conf_threshold=thr, **kw)


def test_threshold_limits():
    w = synth.make_weights(_conf_dims(0.0), seed=21)
    prompt = synth.make_prompts(_conf_dims(0.0), 1, 6, 6, seed=5)[0]
    mc = [synth.interleave(g, 1, 4) for g in range(15)]
    mods, ctrs = [m for m, _ in mc], [c for _, c in mc]
    # threshold 0: an entropy is never below it, every step runs all layers = plain decoding
    _, _, a = _run_dyn(_conf_dims(0.0), w, prompt, mods, ctrs)
    plain = bf.decode_stream(synth.model_dims(MICRO, 5, 1, 0), w, prompt, mods, ctrs)
    assert all(g["depth"] == 5 for g in a)
    assert [g["token"] for g in a] == [x["token"] for x in plain]
    # infinite threshold: every speech step leaves at the start layer (fixed-layer exit), text runs all layers
    _, _, b = _run_dyn(_conf_dims(float("inf")), w, prompt, mods, ctrs)
    assert [g["depth"] for g in b] == [5 if m == 0 else 2 for m in mods]
    fixed = bf.decode_stream(_conf_dims(0.0), w, prompt, mods, ctrs, depths=[5 if m == 0 else 2 for m in mods])
    assert [g["token"] for g in b] == [x["token"] for x in fixed]


@pytest.mark.parametrize("conf_mods,text_exit", [(2, 0), (1, 0), (3, 0)])
def test_confidence_rule_equals_cache_free_recomputation(conf_mods, text_exit):
    """Thresholds placed inside the range of entropies the random heads produce, so that exits
    happen at several different layers; the modality that is not decided by confidence follows
    the periodic schedule (Sec. V-E row G11 pairs confidence on text with Even on speech)."""
    base = _conf_dims(0.0, start=2, mods=conf_mods, text_exit=text_exit)
    w = synth.make_weights(base, seed=33)
    prompt = synth.make_prompts(base, 1, 6, 6, seed=8)[0]
    mc = [synth.interleave(g, 2, 4) for g in range(24)]
    mods, ctrs = [m for m, _ in mc], [c for _, c in mc]
    # entropies at full depth tell where a useful threshold lies (medians per modality)
    _, _, probe = _run_dyn(base, w, prompt, mods, ctrs)
    ents = sorted(e for g in probe for e in g["entropies"] if e >= 0)
    assert ents
    thr = ents[len(ents) // 2] + 1e-6
    dims = dict(base, conf_threshold=thr)
    _, _, got = _run_dyn(dims, w, prompt, mods, ctrs)
    ref = bf.decode_stream(dims, w, prompt, mods, ctrs)
    # no entropy of the run may sit on the threshold, or two correct programs could disagree
    for x in ref:
        assert all(abs(e - thr) > 1e-9 for e in x["entropies"].values())
    assert [g["depth"] for g in got] == [x["depth"] for x in ref]
    assert [g["token"] for g in got] == [x["token"] for x in ref]
    for g, x in zip(got, ref):
        np.testing.assert_allclose(g["hidden"], x["hidden"], rtol=1e-9, atol=1e-11)
        for l, e in x["entropies"].items():
            assert abs(g["entropies"][l - 1] - e) < 1e-9
    depths = [g["depth"] for g in got]
    conf_depths = {d for d, m in zip(depths, mods) if (conf_mods >> m) & 1}
    assert len(conf_depths) >= 2, depths           # exits at more than one layer
    for d, m, c in zip(depths, mods, ctrs):        # the other modality keeps the schedule (e = 3, K = 2)
        if not (conf_mods >> m) & 1:
            assert d == (5 if (m == 0 or c % 2 == 0) else 3)

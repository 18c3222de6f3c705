"""GPU parity at the full model shapes of the five workloads (launch configuration of bench.py).

The oracle cannot afford prompts of many hundreds of tokens at these shapes, so the workload runs
start from a cache of stand-in values (synth.synth_kv) loaded into both sides; from there the
library and the oracle run the same interleaved steps, teacher-forced on the oracle's tokens.
Real prefill at these shapes is compared on prompts of 131 tokens (two full chunks of 64 rows and
a ragged third).
With a batch the oracle follows a seeded subset of the sequences (sequences are independent,
which the small-shape tests establish); the other sequences run free and are held to the exit
schedule only.  Acceptance rules are those of parity_util: depths bit-exact, hidden states and
logits within 2e-2, tokens identical where the oracle's top-2 margin exceeds 5e-2."""
import numpy as np
import pytest
import torch

from paper_2603_09215_b200 import synth

pytestmark = pytest.mark.gpu


def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")


class Model:
    """Random weights of a shape, once per module, on the host and on the device."""

    def __init__(self, shape, head_layers):
        from paper_2603_09215_b200 import binding
        self.shape = shape
        self.dims0 = synth.model_dims(shape, head_layers[0], 1, 0)
        self.w = synth.make_weights(self.dims0, seed=0, head_layers=head_layers)
        self.gw = binding.upload_weights(self.w)


@pytest.fixture(scope="module")
def step_model():
    _need_gpu()
    m = Model("step", [20, 26, 27, 28])
    yield m
    del m.gw
    torch.cuda.empty_cache()


@pytest.fixture(scope="module")
def glm_model():
    _need_gpu()
    m = Model("glm", [20, 30, 40])
    yield m
    del m.gw
    torch.cuda.empty_cache()


def _load_cache(P, lens, checked, dims, shared_seed=77):
    """Stand-in cache of lens[s] positions for every slot; the checked slots get their own
    values (also given to their oracle), the others share one set."""
    from oracle.bruteforce import bf16_to_f64
    L = dims["n_layers"]
    n_max = max(lens)
    shared_k, shared_v = synth.synth_kv(dims, n_max, seed=shared_seed)
    # stand-in values are bf16 bit patterns; the cache holds fp16, which represents them exactly
    dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16).to(torch.float16)
    for layer in range(1, L + 1):
        kt, vt = dev(shared_k[layer - 1]), dev(shared_v[layer - 1])
        for s, n in enumerate(lens):
            if s not in checked:
                P.g.import_kv(s, layer, 0, kt[:n], vt[:n])
    for s in checked:
        k, v = synth.synth_kv(dims, lens[s], seed=1000 + s)
        for layer in range(1, L + 1):
            P.g.import_kv(s, layer, 0, dev(k[layer - 1]), dev(v[layer - 1]))
            kf, vf = bf16_to_f64(k[layer - 1]), bf16_to_f64(v[layer - 1])
            for p in range(lens[s]):
                P.os[s].set_kv(layer, p, kf[p], vf[p])
        P.os[s].set_len(lens[s])
    for s, n in enumerate(lens):
        P.g.set_len(s, n)
    torch.cuda.synchronize()


def _run(model, wl_name, steps, g0, n_checked, lens=None, exit_layer=None, period=None, batch=None):
    from tests import parity_util as pu
    wl = dict(synth.WORKLOADS[wl_name])
    e = wl["exit_layer"] if exit_layer is None else exit_layer
    K = wl["refresh_period"] if period is None else period
    dims = synth.model_dims(model.shape, e, K, wl["refresh_phase"])
    B = wl["batch"] if batch is None else batch
    rng = np.random.Generator(np.random.PCG64(5))
    if lens is None:
        lens = [int(x) for x in rng.integers(wl["prompt"][0], wl["prompt"][1] + 1, size=B)] if wl["prompt"][0] != wl["prompt"][1] \
            else [wl["prompt"][0] - 1] * B
    phi, off = synth.make_phases(B, wl["n_text"], wl["n_speech"], K, wl["random_phase"], seed=3)
    checked = sorted(int(x) for x in rng.choice(B, size=min(n_checked, B), replace=False))
    P = pu.Pair(dims, model.w, B, max(lens) + steps + 2, max(K - 1, 1), oracle_slots=checked, gw=model.gw)
    _load_cache(P, lens, set(checked), dims)
    V = dims["vocab_text"] + dims["vocab_speech"]
    P.next_in = [int(x) for x in rng.integers(0, V, size=B)]
    mixed = 0
    for g in range(g0, g0 + steps):
        mc = [synth.interleave(g, wl["n_text"], wl["n_speech"], int(p), int(o)) for p, o in zip(phi, off)]
        _, _, dep = P.step([m for m, _ in mc], [c for _, c in mc])
        mixed += len(set(int(x) for x in dep)) > 1
    stats = dict(P.stats, mixed_steps=mixed, checked=checked)
    P.close()
    return stats


def test_config2_step_shape_batch1(step_model):
    """Workload 2: Step-shaped, batch 1, cache of 511 positions, the first 256 decode steps of
    the workload's 1024 (51 interleave cycles: text, refresh, three early exits; every cycle's
    text step pushes three pending rows through the upper layers with its own)."""
    st = _run(step_model, "cfg2_step_b1", steps=256, g0=0, n_checked=1)
    print("cfg2", st)
    assert st["steps"] == 256 and st["tok_checked"] >= 128
    assert st["max_flush"] == 3 and st["flushes"] >= 50


def test_config3_step_shape_batch64(step_model):
    """Workload 3: batch 64, ragged caches of 256..2048 positions, random interleave phases and
    counter offsets so every step mixes depths; the oracle follows two of the sequences for two
    interleave cycles."""
    st = _run(step_model, "cfg3_step_b64", steps=10, g0=0, n_checked=2)
    print("cfg3", st)
    assert st["mixed_steps"] >= 8
    assert st["flushes"] >= 2


def test_config4_glm_shape_batch16(glm_model):
    """Workload 4: GLM-shaped, batch 16, caches of 1023 positions, phase-aligned 13:26 interleave,
    two whole interleave cycles (78 steps): text chunks, refreshes every fourth speech position
    with three pending rows each, and the text step after a chunk that ends on an early exit."""
    st = _run(glm_model, "cfg4_glm_b16", steps=78, g0=0, n_checked=2)
    print("cfg4", st)
    assert st["steps"] == 78 and st["max_flush"] == 3 and st["flushes"] >= 24


def test_config5_glm_shape_long_context(glm_model):
    """Workload 5 (long-context stress): caches of 8191 positions; batch 128 with the oracle on
    two sequences, for the e=30, K=4 cell, two whole interleave cycles (78 steps) with random
    phases, so the checked sequences refresh with three pending rows while others sit at any
    other point of their cycle."""
    st = _run(glm_model, "cfg5_glm_b128", steps=78, g0=0, n_checked=2, lens=[8191] * 128)
    print("cfg5", st)
    assert st["steps"] == 78 and st["max_flush"] == 3 and st["flushes"] >= 20


def _real_prefill(model, wl_name, prompt_len):
    """A prompt long enough for two full 64-row prefill chunks and a ragged third, ingested by
    sparsk_prefill (the tcgen05 GEMMs and the tcgen05 attention kernel at blocks of hundreds of
    query vectors per kv head) and by the oracle; the cache of every layer is compared, then one
    interleave cycle runs on top of it."""
    from tests import parity_util as pu
    wl = synth.WORKLOADS[wl_name]
    dims = synth.model_dims(model.shape, wl["exit_layer"], wl["refresh_period"], wl["refresh_phase"])
    K = wl["refresh_period"]
    cyc = wl["n_text"] + wl["n_speech"]
    prompt = synth.make_prompts(dims, 1, prompt_len, prompt_len, seed=21)[0]
    P = pu.Pair(dims, model.w, 1, prompt_len + cyc + 3, max(K - 1, 1), prefill_rows=64, gw=model.gw)
    P.prefill([prompt])
    assert P.g.slot_state(0) == (prompt_len - 1, 0)
    P.check_cache(0, range(1, dims["n_layers"] + 1), prompt_len - 1)
    for g in range(cyc + 1):       # one whole cycle and the text step that follows it (it flushes the chunk's tail)
        m, c = synth.interleave(g, wl["n_text"], wl["n_speech"])
        P.step([m], [c])
    ln, pend = P.g.slot_state(0)
    P.check_cache(0, range(1, dims["exit_layer"] + 1), ln)
    P.check_cache(0, range(dims["exit_layer"] + 1, dims["n_layers"] + 1), ln - pend)
    st = dict(P.stats)
    P.close()
    return st


def test_real_prefill_step_shape(step_model):
    st = _real_prefill(step_model, "cfg2_step_b1", 131)
    print("prefill step", st)
    assert st["steps"] == 6 and st["max_flush"] == 3


def test_real_prefill_glm_shape(glm_model):
    st = _real_prefill(glm_model, "cfg4_glm_b16", 131)
    print("prefill glm", st)
    assert st["steps"] == 40 and st["max_flush"] == 3


@pytest.mark.parametrize("e", [20, 30, 40])
@pytest.mark.parametrize("K", [2, 4, 8])
def test_config5_sweep_depths(glm_model, e, K):
    """Every (e, K) cell of workload 5's sweep: exit depths of all 128 sequences over one
    interleave cycle are exactly the schedule's (checked inside the driver for every step)."""
    st = _run(glm_model, "cfg5_glm_b128", steps=39, g0=0, n_checked=0, lens=[64] * 128, exit_layer=e, period=K)
    assert st["steps"] == 39


def test_confidence_exit_step_shape(step_model):
    """Confidence-based exit (Sec. V-B) at the Step shape with the paper's start layer for that
    backbone (row S3: layer 26) on speech steps, from a stand-in cache of 511 positions.  With the
    paper's threshold 0.1 random heads are never confident (their entropy is near ln 6561): every
    speech step pays for the heads of layers 26 and 27 and runs all 28 layers, the wasted
    projection of Sec. V-C.  With an infinite threshold every speech step leaves at layer 26 and
    the next text step carries the pending positions through layers 27 and 28."""
    from oracle import oracle as ora
    from tests import parity_util as pu
    from paper_2603_09215_b200 import binding
    for thr, want_speech in ((0.1, 28), (float("inf"), 26)):
        dims = synth.model_dims("step", 20, 4, 0, conf_modalities=2, conf_start=26, conf_threshold=thr)
        g = binding.Sparsk(dims, step_model.gw, 1, 511 + 16, 8)
        om = ora.OracleModel(dims, step_model.w, max_len=511 + 16)
        sq = om.new_seq(8)
        k, v = synth.synth_kv(dims, 511, seed=1000)
        from oracle.bruteforce import bf16_to_f64
        dev = lambda a: torch.from_numpy(a.view(np.int16)).cuda().view(torch.bfloat16).to(torch.float16)
        for layer in range(1, 29):
            g.import_kv(0, layer, 0, dev(k[layer - 1]), dev(v[layer - 1]))
            kf, vf = bf16_to_f64(k[layer - 1]), bf16_to_f64(v[layer - 1])
            for p in range(511):
                sq.set_kv(layer, p, kf[p], vf[p])
        g.set_len(0, 511)
        sq.set_len(511)
        V, Vt = dims["vocab_text"] + dims["vocab_speech"], dims["vocab_text"]
        dbg_h = torch.zeros((1, dims["d_model"]), dtype=torch.float32, device="cuda")
        dbg_z = torch.zeros((1, V), dtype=torch.float32, device="cuda")
        g.set_debug(dbg_h, dbg_z)
        tok = torch.tensor([1234], dtype=torch.int32, device="cuda")
        ot, od = torch.zeros(1, dtype=torch.int32, device="cuda"), torch.zeros(1, dtype=torch.int32, device="cuda")
        nxt = 1234
        for step in range(7):
            m, c = synth.interleave(step, 1, 4)
            tok[0] = nxt
            g.decode_step([0], tok, [m], [c], ot, od)
            g.check()
            dep = int(od.cpu()[0])
            assert dep == (28 if m == 0 else want_speech), (step, m, dep)
            r = sq.decode_step_dyn(nxt, m, c, forced_depth=dep)
            ent = g.conf_entropies(1)[0]
            for l in (26, 27):
                if m == 1 and l <= dep and l < 28:
                    assert abs(float(ent[l]) - r["entropies"][l - 1]) <= 1e-3, (l, ent[l], r["entropies"][l - 1])
                    assert (float(ent[l]) < thr) == (l == dep)
            lo, hi = (0, Vt) if m == 0 else (Vt, V)
            H, Z = dbg_h.cpu().numpy().astype(np.float64)[0], dbg_z.cpu().numpy().astype(np.float64)[0]
            assert pu.rel_err(H, r["hidden"]) <= pu.REL_TOL
            assert pu.rel_err(Z[lo:hi], r["logits"][lo:hi]) <= pu.REL_TOL
            if r["margin"] > pu.MARGIN:
                assert int(ot.cpu()[0]) == r["token"]
            nxt = r["token"]
            assert g.slot_state(0) == (sq.len, len(sq.pending))
        g.close()

"""GPU parity of confidence-based early exit (Sec. V-B, compared method 3) against the oracle.

The depth of a confidence step is decided by comparing an entropy with a threshold, a
floating-point decision the two sides take on logits that differ in the last digits.  So the
library decides, its entropies are compared with the oracle's own (tolerance below), the depth
it chose must be the one its entropies imply, and the oracle is then told that depth and must
reproduce the step's hidden state, logits and token under the usual rules.  Where the oracle's
entropies are farther from the threshold than the tolerance the two decisions are necessarily
the same; the test counts those."""
import numpy as np
import pytest
import torch

from paper_2603_09215_b200 import synth

pytestmark = pytest.mark.gpu

ENT_TOL = 3e-4     # entropies: absolute, nats.  An entropy is far less sensitive than a logit: near the
                   # flat distributions random heads give, an error dz of the logits moves it by about
                   # dz * std(z) / sqrt(ids), i.e. 1e-5 here; measured deviations are printed below.


@pytest.fixture(scope="module")
def util():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity_util
    return parity_util


def _probe_threshold(dims, w, prompt, mods, ctrs):
    """A threshold in the middle of the entropies the random heads produce (oracle at threshold 0)."""
    from oracle import oracle as ora
    m = ora.OracleModel(dict(dims, conf_threshold=0.0), w, max_len=len(prompt) + len(mods) + 2)
    s = m.new_seq(64)
    s.prefill(prompt[:-1])
    tok = int(prompt[-1])
    ents = []
    for mod, c in zip(mods, ctrs):
        r = s.decode_step_dyn(tok, mod, c)
        ents += [e for e in r["entropies"] if e >= 0]
        tok = r["token"]
    ents.sort()
    return ents[len(ents) // 2] + 1e-5


@pytest.mark.parametrize("conf_mods,options", [(2, {}), (1, {}), (3, {"mega": 0}), (2, {"mega": 0, "gemm_min_rows": 1}),
                                               (2, {"mega": 0, "gemm_min_rows": 1 << 30})])
def test_confidence_exit_matches_oracle(util, conf_mods, options):
    from oracle import oracle as ora
    from paper_2603_09215_b200 import binding
    base = synth.model_dims("tiny", 2, 2, 0, conf_modalities=conf_mods, conf_start=1, conf_threshold=0.0)
    w = synth.make_weights(base, seed=0)
    B, steps, nt, ns = 3, 36, 2, 5
    prompts = synth.make_prompts(base, B, 9, 30, seed=31)
    phases = [0, 3, 5]
    sched = [[synth.interleave(g, nt, ns, ph) for ph in phases] for g in range(steps)]
    thr = _probe_threshold(base, w, prompts[0], [mc[0][0] for mc in sched], [mc[0][1] for mc in sched])
    dims = dict(base, conf_threshold=thr)
    L, V, Vt = dims["n_layers"], dims["vocab_text"] + dims["vocab_speech"], dims["vocab_text"]
    max_len = 30 + steps + 2
    gw = binding.upload_weights(w)
    g = binding.Sparsk(dims, gw, B, max_len, 16, prefill_rows=16)
    for k, v in options.items():
        g.set_option(k, v)
    om = ora.OracleModel(dims, w, max_len=max_len)
    seqs = [om.new_seq(16) for _ in range(B)]
    g.prefill(list(range(B)), [p[:-1] for p in prompts])
    for s, p in zip(seqs, prompts):
        s.prefill(p[:-1])
    dbg_h = torch.zeros((B, dims["d_model"]), dtype=torch.float32, device="cuda")
    dbg_z = torch.zeros((B, V), dtype=torch.float32, device="cuda")
    g.set_debug(dbg_h, dbg_z)
    tok = torch.tensor([int(p[-1]) for p in prompts], dtype=torch.int32, device="cuda")
    out_tok = torch.zeros(B, dtype=torch.int32, device="cuda")
    out_dep = torch.zeros(B, dtype=torch.int32, device="cuda")
    nxt = [int(p[-1]) for p in prompts]
    clear = unclear = early = 0
    max_dev = 0.0
    depths_seen = set()
    for mc in sched:
        mods, ctrs = [m for m, _ in mc], [c for _, c in mc]
        tok[:] = torch.tensor(nxt, dtype=torch.int32)
        g.decode_step(list(range(B)), tok, mods, ctrs, out_tok, out_dep)
        g.check()
        got_tok, got_dep = out_tok.cpu().numpy(), out_dep.cpu().numpy()
        ent_gpu = g.conf_entropies(B)
        H, Z = dbg_h.cpu().numpy().astype(np.float64), dbg_z.cpu().numpy().astype(np.float64)
        for i in range(B):
            dep = int(got_dep[i])
            by_conf = (conf_mods >> mods[i]) & 1
            r = seqs[i].decode_step_dyn(nxt[i], mods[i], ctrs[i], forced_depth=dep)
            if by_conf:
                # the library's own entropies imply the depth it chose ...
                for l in range(1, L):
                    eg = float(ent_gpu[i, l])
                    if l < dep or (l == dep and dep < L):
                        assert eg >= 0 and abs(eg - r["entropies"][l - 1]) <= ENT_TOL, (i, l, eg, r["entropies"][l - 1])
                        max_dev = max(max_dev, abs(eg - r["entropies"][l - 1]))
                        assert (eg < thr) == (l == dep), (i, l, dep, eg, thr)
                    else:
                        assert eg == -1.0, (i, l, dep, eg)
                # ... and where the oracle's are clear of the threshold it agrees by itself
                own = [e for e in r["entropies"][:dep if dep < L else L - 1] if e >= 0]
                if all(abs(e - thr) > ENT_TOL for e in own):
                    clear += 1
                else:
                    unclear += 1
                early += dep < L
                depths_seen.add(dep)
            else:
                want = L if (mods[i] == 0 or ctrs[i] % 2 == 0) else 2     # text_exit 0, Even, e = 2
                assert dep == want, (i, dep, want)
            eh = util.rel_err(H[i], r["hidden"])
            lo, hi = (0, Vt) if mods[i] == 0 else (Vt, V)
            ez = util.rel_err(Z[i][lo:hi], r["logits"][lo:hi])
            assert eh <= util.REL_TOL and ez <= util.REL_TOL, (i, dep, eh, ez)
            assert np.isneginf(np.delete(Z[i], np.s_[lo:hi])).all()
            assert got_tok[i] == lo + int(np.argmax(Z[i][lo:hi]))
            if r["margin"] > util.MARGIN:
                assert got_tok[i] == r["token"]
            nxt[i] = r["token"]
            assert g.slot_state(i) == (seqs[i].len, len(seqs[i].pending))
    print("confidence", dict(clear=clear, unclear=unclear, early=early, depths=sorted(depths_seen), max_entropy_dev=max_dev))
    assert clear > 3 * max(1, unclear) and early >= 5 and len(depths_seen) >= 3
    # the cache: every position complete up to the layer it has been carried to
    for i in range(B):
        ln = seqs[i].len
        fill = dict(zip(seqs[i].pending, seqs[i].pending_fill))
        for layer in range(1, L + 1):
            k, v = g.export_kv(i, layer, 0, ln)
            k, v = k.float().cpu().numpy().astype(np.float64), v.float().cpu().numpy().astype(np.float64)
            for p in range(ln):
                if fill.get(p, L) >= layer:
                    rk, rv = seqs[i].get_kv(layer, p)
                    assert util.rel_err(k[p], rk) <= util.REL_TOL and util.rel_err(v[p], rv) <= util.REL_TOL, (i, layer, p)
    g.close()


def test_confidence_dims_and_heads_are_checked(util):
    from paper_2603_09215_b200 import binding
    base = synth.model_dims("tiny", 2, 2, 0, conf_modalities=2, conf_start=2, conf_threshold=0.5)
    w = synth.make_weights(base, seed=0, head_layers=[2, 4])        # layer 3 has no head
    gw = binding.upload_weights(w)
    with pytest.raises(binding.SparskError) as ei:
        binding.Sparsk(base, gw, 1, 32, 4)
    assert ei.value.code == binding.ENOHEAD
    for bad in (dict(conf_start=0), dict(conf_start=4), dict(conf_modalities=4), dict(conf_threshold=-1.0)):
        with pytest.raises(binding.SparskError) as ei:
            binding.Sparsk(dict(base, **bad), gw, 1, 32, 4)
        assert ei.value.code == binding.EINVAL, bad

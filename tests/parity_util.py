"""Shared driver of the GPU-vs-oracle parity tests: runs the CUDA library and the C oracle on the
same seeded inputs, teacher-forced on the oracle's token stream, and applies the acceptance
rules: exit depths bit-exact; every exited hidden state and (restricted) logit vector within
2e-2 max error relative to the vector's largest magnitude; greedy token identical wherever the
oracle's top-2 margin exceeds 5e-2."""
import numpy as np
import torch

from oracle import oracle as ora
from paper_2603_09215_b200 import binding, synth

REL_TOL = 2e-2      # bf16 storage of weights/activations/cache against the fp64 oracle
MARGIN = 5e-2


def rel_err(got: np.ndarray, ref: np.ndarray) -> float:
    return float(np.abs(got - ref).max() / max(np.abs(ref).max(), 1e-30))


class Pair:
    """A CUDA context and one oracle sequence per slot, fed the same inputs."""

    def __init__(self, dims, weights, n_seqs, max_seq_len, max_pending, prefill_rows=0, heads=None,
                 options=None, oracle_slots=None, gw=None):
        """oracle_slots: the slots that get an oracle sequence and are checked (default: all);
        the other slots run free on the library's own tokens.  gw: weights already on the device."""
        self.dims = dims
        self.w = weights
        self.gw = gw if gw is not None else binding.upload_weights(weights)
        self.g = binding.Sparsk(dims, self.gw, n_seqs, max_seq_len, max_pending, prefill_rows)
        for k, v in (options or {}).items():
            self.g.set_option(k, v)
        self.om = ora.OracleModel(dims, weights, max_len=max_seq_len)
        self.checked = set(range(n_seqs)) if oracle_slots is None else set(oracle_slots)
        self.os = [self.om.new_seq(max(1, max_pending)) if s in self.checked else None for s in range(n_seqs)]
        self.n = n_seqs
        V = dims["vocab_text"] + dims["vocab_speech"]
        self.dbg_h = torch.zeros((n_seqs, dims["d_model"]), dtype=torch.float32, device="cuda")
        self.dbg_z = torch.zeros((n_seqs, V), dtype=torch.float32, device="cuda")
        self.g.set_debug(self.dbg_h, self.dbg_z)
        self.tok = torch.zeros(n_seqs, dtype=torch.int32, device="cuda")
        self.out_tok = torch.zeros(n_seqs, dtype=torch.int32, device="cuda")
        self.out_dep = torch.zeros(n_seqs, dtype=torch.int32, device="cuda")
        self.stats = {"steps": 0, "max_hidden": 0.0, "max_logit": 0.0, "tok_checked": 0,
                      "tok_skipped": 0, "max_flush": 0, "flushes": 0}

    def prefill(self, prompts):
        """prompts: full prompts; the last token of each is kept as the first step's input."""
        self.g.prefill(list(range(self.n)), [p[:-1] for p in prompts])
        self.g.check()
        for s, p in zip(self.os, prompts):
            if s is not None:
                s.prefill(p[:-1])
        self.next_in = [int(p[-1]) for p in prompts]

    def step(self, mods, ctrs, slots=None):
        slots = list(range(self.n)) if slots is None else list(slots)
        k = len(slots)
        pend_before = [len(self.os[s].pending) if s in self.checked else 0 for s in slots]
        ref = [self.os[s].decode_step(self.next_in[s], mods[i], ctrs[i]) if s in self.checked else None
               for i, s in enumerate(slots)]
        self.tok[:k] = torch.tensor([self.next_in[s] for s in slots], dtype=torch.int32)
        self.g.decode_step(slots, self.tok, mods, ctrs, self.out_tok, self.out_dep)
        self.g.check()
        got_tok = self.out_tok[:k].cpu().numpy()
        got_dep = self.out_dep[:k].cpu().numpy()
        # hidden states and logits of the checked sequences only (a logit row is ~0.7 MB)
        rows = [i for i, s in enumerate(slots) if s in self.checked]
        sel = torch.tensor(rows, dtype=torch.long, device="cuda")
        H = dict(zip(rows, self.dbg_h[sel].cpu().numpy().astype(np.float64)))
        Z = dict(zip(rows, self.dbg_z[sel].cpu().numpy().astype(np.float64)))
        Vt = self.dims["vocab_text"]
        V = Vt + self.dims["vocab_speech"]
        L, e, K, r_ = (self.dims[k] for k in ("n_layers", "exit_layer", "refresh_period", "refresh_phase"))
        for i, s in enumerate(slots):
            r = ref[i]
            if r is None:
                # unchecked sequence: its depth still has to follow the schedule; it runs on
                # the token the library produced
                te = self.dims.get("text_exit", 0)
                Km, rm = (self.dims["text_period"], self.dims.get("text_phase", 0)) \
                    if mods[i] == 0 and self.dims.get("text_period", 0) > 0 else (K, r_)
                want = L if ((mods[i] == 0 and te == 0) or (mods[i] == 1 and te == 2)) else (L if ctrs[i] % Km == rm else e)
                assert got_dep[i] == want, (i, got_dep[i], want)
                self.next_in[s] = int(got_tok[i])
                continue
            assert got_dep[i] == r["depth"], (i, got_dep[i], r["depth"])
            if r["depth"] == L and e < L and pend_before[i]:
                # a full-depth step that pushed pending rows through the upper layers with its own
                self.stats["flushes"] += 1
                self.stats["max_flush"] = max(self.stats["max_flush"], pend_before[i])
            eh = rel_err(H[i], r["hidden"])
            lo, hi = (0, Vt) if mods[i] == 0 else (Vt, V)
            ez = rel_err(Z[i][lo:hi], r["logits"][lo:hi])
            assert eh <= REL_TOL, f"seq {s} step {self.stats['steps']}: hidden rel err {eh:.3e}"
            assert ez <= REL_TOL, f"seq {s} step {self.stats['steps']}: logit rel err {ez:.3e}"
            assert np.isneginf(np.delete(Z[i], np.s_[lo:hi])).all()
            assert lo <= got_tok[i] < hi
            # the emitted token is the arg max of the library's own logits (lowest id on ties)
            assert got_tok[i] == lo + int(np.argmax(Z[i][lo:hi]))
            if r["margin"] > MARGIN:
                assert got_tok[i] == r["token"], (s, got_tok[i], r["token"], r["margin"])
                self.stats["tok_checked"] += 1
            else:
                self.stats["tok_skipped"] += 1
            self.stats["max_hidden"] = max(self.stats["max_hidden"], eh)
            self.stats["max_logit"] = max(self.stats["max_logit"], ez)
            self.next_in[s] = r["token"]          # teacher forcing on the oracle's stream
        self.stats["steps"] += 1
        return ref, got_tok, got_dep

    def check_cache(self, slot, layers, upto):
        """Cached K/V of `slot` for positions [0, upto) against the oracle's (Sec. IV-B.3 invariant)."""
        for layer in layers:
            k, v = self.g.export_kv(slot, layer, 0, upto)
            k = k.float().cpu().numpy().astype(np.float64)
            v = v.float().cpu().numpy().astype(np.float64)
            rk = np.stack([self.os[slot].get_kv(layer, p)[0] for p in range(upto)])
            rv = np.stack([self.os[slot].get_kv(layer, p)[1] for p in range(upto)])
            assert rel_err(k, rk) <= REL_TOL, (layer, rel_err(k, rk))
            assert rel_err(v, rv) <= REL_TOL, (layer, rel_err(v, rv))

    def close(self):
        self.g.close()


def schedule(wl_or_none, steps, n_text, n_speech, phases, offsets):
    out = []
    for g in range(steps):
        mc = [synth.interleave(g, n_text, n_speech, int(ph), int(of)) for ph, of in zip(phases, offsets)]
        out.append(([m for m, _ in mc], [c for _, c in mc]))
    return out

"""Seeded synthetic inputs: model shapes, random weights, prompts, interleave bookkeeping.

This module holds no arithmetic of the decoding method.  It only draws random
numbers, rounds weights once to bfloat16, and lays out which generated token is text
or speech (Sec. III: N_text text tokens then N_speech speech tokens, repeated) and
what its index inside its chunk is.  Both the CUDA binding's callers and the CPU
checkers take their inputs from here.

Weights are returned as NumPy ``uint16`` arrays of bfloat16 bit patterns:
matrices, embeddings and head projections ~ N(0, 0.02); norm gains ~ 1 + N(0, 0.02).
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

# Model shapes.  "step" follows a 28-layer 7B-class backbone with a 1:4 text:speech
# interleave, "glm" a 40-layer 9B-class backbone with 13:26 (Sec. V-A); "tiny" is
# the small case a CPU finishes in seconds.
SHAPES = {
    "tiny": dict(n_layers=4, d_model=256, n_q_heads=4, n_kv_heads=2, head_dim=64, d_ffn=688,
                 vocab_text=1024, vocab_speech=512, rms_eps=1e-6, rope_base=10000.0),
    "step": dict(n_layers=28, d_model=3584, n_q_heads=28, n_kv_heads=4, head_dim=128,
                 d_ffn=18944, vocab_text=151936, vocab_speech=6561, rms_eps=1e-6,
                 rope_base=10000.0),
    "glm": dict(n_layers=40, d_model=4096, n_q_heads=32, n_kv_heads=2, head_dim=128,
                d_ffn=13696, vocab_text=151552, vocab_speech=16384, rms_eps=1e-6,
                rope_base=10000.0),
}
# Cut-down copies for profiler captures: the layers keep the full shapes (one layer's weights are
# still several times the L2), but only four of them and a short text vocabulary, so that the
# whole model stays near 2 GB on the device.
SHAPES["step4"] = dict(SHAPES["step"], n_layers=4, vocab_text=8192)
SHAPES["glm4"] = dict(SHAPES["glm"], n_layers=4, vocab_text=8192)

# Workloads: (shape, batch, prompt length(s), decode steps, N_text, N_speech, e, K, r).
WORKLOADS = {
    "cfg1_tiny_b1": dict(shape="tiny", batch=1, prompt=(32, 32), steps=96, n_text=2, n_speech=4,
                         exit_layer=2, refresh_period=3, refresh_phase=0, random_phase=False),
    "cfg2_step_b1": dict(shape="step", batch=1, prompt=(512, 512), steps=1024, n_text=1,
                         n_speech=4, exit_layer=20, refresh_period=4, refresh_phase=0,
                         random_phase=False),
    "cfg3_step_b64": dict(shape="step", batch=64, prompt=(256, 2048), steps=512, n_text=1,
                          n_speech=4, exit_layer=20, refresh_period=4, refresh_phase=0,
                          random_phase=True),
    "cfg4_glm_b16": dict(shape="glm", batch=16, prompt=(1024, 1024), steps=2048, n_text=13,
                         n_speech=26, exit_layer=30, refresh_period=4, refresh_phase=0,
                         random_phase=False),
    "cfg5_glm_b128": dict(shape="glm", batch=128, prompt=(8192, 8192), steps=256, n_text=13,
                          n_speech=26, exit_layer=30, refresh_period=4, refresh_phase=0,
                          random_phase=True),
    # profiler-sized cases (not benchmark lines)
    "prof_step4_b1": dict(shape="step4", batch=1, prompt=(512, 512), steps=64, n_text=1, n_speech=4,
                          exit_layer=2, refresh_period=4, refresh_phase=0, random_phase=False),
    "prof_step4_b64": dict(shape="step4", batch=64, prompt=(256, 512), steps=64, n_text=1, n_speech=4,
                           exit_layer=2, refresh_period=4, refresh_phase=0, random_phase=True),
    "prof_step4_b64_ragged": dict(shape="step4", batch=64, prompt=(256, 2048), steps=64, n_text=1, n_speech=4,
                                  exit_layer=2, refresh_period=4, refresh_phase=0, random_phase=True),
    "prof_glm4_b128": dict(shape="glm4", batch=128, prompt=(8192, 8192), steps=64, n_text=13,
                           n_speech=26, exit_layer=3, refresh_period=4, refresh_phase=0,
                           random_phase=True),
    "prof_glm4_b16": dict(shape="glm4", batch=16, prompt=(1024, 1024), steps=64, n_text=13,
                          n_speech=26, exit_layer=3, refresh_period=4, refresh_phase=0,
                          random_phase=False),
}

PER_LAYER = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down",
             "head_norm", "head_proj")


def model_dims(shape: str, exit_layer: int, refresh_period: int, refresh_phase: int = 0,
               text_exit: int = 0, **over) -> dict:
    d = dict(SHAPES[shape]) if isinstance(shape, str) else dict(shape)
    d.update(exit_layer=exit_layer, refresh_period=refresh_period, refresh_phase=refresh_phase,
             text_exit=text_exit)
    d.update(over)
    return d


def _draw(seed: int, idx: int, shape, mean: float) -> np.ndarray:
    g = torch.Generator("cpu")
    g.manual_seed(seed * 1_000_003 + idx)
    t = torch.empty(shape, dtype=torch.float32).normal_(mean, 0.02, generator=g)
    return t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)


def make_weights(dims: dict, seed: int = 0, head_layers=None, threads: int = 8) -> dict:
    """Random weights for `dims`.  `head_layers`: iterable of 1-based layers that get an exit
    head (default: every layer); the others are None."""
    L, d = dims["n_layers"], dims["d_model"]
    Hq, Hkv, hd, F = dims["n_q_heads"], dims["n_kv_heads"], dims["head_dim"], dims["d_ffn"]
    V = dims["vocab_text"] + dims["vocab_speech"]
    heads = set(range(1, L + 1)) if head_layers is None else set(int(x) for x in head_layers)
    shapes = {"attn_norm": (d,), "wq": (Hq * hd, d), "wk": (Hkv * hd, d), "wv": (Hkv * hd, d),
              "wo": (d, Hq * hd), "mlp_norm": (d,), "w_gate": (F, d), "w_up": (F, d),
              "w_down": (d, F), "head_norm": (d,), "head_proj": (V, d)}
    jobs = [("embed", None, 0, (V, d), 0.0)]
    for l in range(L):
        for j, name in enumerate(PER_LAYER):
            if name.startswith("head") and (l + 1) not in heads:
                continue
            mean = 1.0 if name.endswith("norm") else 0.0
            jobs.append((name, l, 1 + l * len(PER_LAYER) + j, shapes[name], mean))
    out = {"embed": None}
    for name in PER_LAYER:
        out[name] = [None] * L
    with ThreadPoolExecutor(max_workers=max(1, threads)) as ex:
        res = list(ex.map(lambda jb: _draw(seed, jb[2], jb[3], jb[4]), jobs))
    for (name, l, _, _, _), arr in zip(jobs, res):
        if l is None:
            out[name] = arr
        else:
            out[name][l] = arr
    return out


def make_prompts(dims: dict, batch: int, lo: int, hi: int, seed: int = 1, len_seed: int = 2):
    """`batch` prompts of uniform random ids over the whole vocabulary; lengths uniform in
    [lo, hi].  Returns a list of int32 arrays."""
    V = dims["vocab_text"] + dims["vocab_speech"]
    gl = np.random.Generator(np.random.PCG64(len_seed))
    lens = gl.integers(lo, hi + 1, size=batch)
    gp = np.random.Generator(np.random.PCG64(seed))
    return [gp.integers(0, V, size=int(n), dtype=np.int32) for n in lens]


def make_phases(batch: int, n_text: int, n_speech: int, refresh_period: int, random_phase: bool,
                seed: int = 3):
    """Per-sequence interleave phase phi_b in [0, N_text+N_speech) and counter offset o_b in
    [0, K); both zero unless `random_phase`."""
    if not random_phase:
        return np.zeros(batch, np.int64), np.zeros(batch, np.int64)
    g = np.random.Generator(np.random.PCG64(seed))
    phi = g.integers(0, n_text + n_speech, size=batch)
    off = g.integers(0, refresh_period, size=batch)
    return phi, off


def interleave(step: int, n_text: int, n_speech: int, phase: int = 0, offset: int = 0,
               running: bool = False):
    """Modality (0 text, 1 speech) of the token generated at index `step`, and its counter.

    Generated index g sits at cycle position u = (g + phase) mod (N_text + N_speech); it is text
    while u < N_text, else speech with in-chunk index j = u - N_text.  The counter handed to the
    schedule is j + offset (restarting at every chunk) or, if `running`, the number of speech
    tokens generated before it plus offset.  Text counters are their in-chunk index."""
    cyc = n_text + n_speech
    u = (step + phase) % cyc
    if u < n_text:
        return 0, u
    j = u - n_text
    if not running:
        return 1, j + offset
    full_cycles, rem = divmod(step + phase, cyc)
    before = full_cycles * n_speech + max(0, rem - n_text)
    first = (phase // cyc) * n_speech + max(0, phase % cyc - n_text)
    return 1, before - first + offset


def make_uniforms(n: int, seed: int) -> np.ndarray:
    """n uniform numbers in [0, 1) as float32 (PCG64): the draws a sampling decoder consumes."""
    g = np.random.Generator(np.random.PCG64(seed))
    u = g.random(n, dtype=np.float32)
    return np.minimum(u, np.float32(0.99999994))


def make_logits(n: int, vocab: int, scale: float, seed: int) -> np.ndarray:
    """[n, vocab] float32 logits ~ N(0, scale): flat distributions for small scales (random heads
    give about 0.3 to 1.3), a few dominant ids for large ones."""
    g = torch.Generator("cpu")
    g.manual_seed(seed)
    return torch.empty((n, vocab), dtype=torch.float32).normal_(0, scale, generator=g).numpy()


def synth_kv(dims: dict, n: int, seed: int) -> tuple:
    """Stand-in cache contents for long-context cases where a real prefill is not affordable on
    the CPU: keys and values ~ N(0, 1) rounded to bfloat16, [L, n, Hkv*hd] uint16 each."""
    L = dims["n_layers"]
    row = dims["n_kv_heads"] * dims["head_dim"]
    g = torch.Generator("cpu")
    g.manual_seed(seed)
    k = torch.empty((L, n, row), dtype=torch.float32).normal_(0, 1, generator=g)
    v = torch.empty((L, n, row), dtype=torch.float32).normal_(0, 1, generator=g)
    cv = lambda t: t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    return cv(k), cv(v)

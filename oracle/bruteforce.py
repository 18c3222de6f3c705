"""Cache-free restatement of what SPAR-K decoding must produce (NumPy, float64).

TEST INFRASTRUCTURE, independent of both the C oracle and the CUDA path.

Sec. IV-B.3 states that every full-depth step restores complete K/V at all layers
for all earlier positions and that an early-exit token is never revised.  Hence the
token emitted at step s, which consumes position p and runs d_s layers, is

    y_s = argmax over the modality's id range of  g_{d_s}( h_p^{(d_s)} )

where h_p^{(l)} are the ordinary causal-transformer hidden states of the token
sequence so far (Sec. III).  This file computes exactly that: a full causal forward
over the whole sequence with no cache and no pending set, once per step.
"""
from __future__ import annotations

import numpy as np


def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def _rms(x, g, eps):
    return x / np.sqrt((x * x).mean(axis=-1, keepdims=True) + eps) * g


def _rope(x, base):
    """x [T, H, hd]; position of row t is t.  Rotate-half pairing (i, i+hd/2)."""
    T, _, hd = x.shape
    half = hd // 2
    inv = base ** (-2.0 * np.arange(half) / hd)
    ang = np.arange(T)[:, None] * inv[None, :]
    c, s = np.cos(ang)[:, None, :], np.sin(ang)[:, None, :]
    a, b = x[..., :half], x[..., half:]
    return np.concatenate([a * c - b * s, b * c + a * s], axis=-1)


def forward_all(dims: dict, w: dict, tokens) -> dict:
    """Full causal forward.  Returns H [L+1, T, d] (H[0] = embeddings, H[l] = h^(l)) and the
    per-layer rotated keys K [L, T, Hkv*hd] and values V [L, T, Hkv*hd]."""
    L, d = dims["n_layers"], dims["d_model"]
    Hq, Hkv, hd = dims["n_q_heads"], dims["n_kv_heads"], dims["head_dim"]
    eps, base = dims["rms_eps"], dims["rope_base"]
    tokens = np.asarray(tokens)
    T = tokens.size
    h = bf16_to_f64(w["embed"])[tokens]
    H = np.empty((L + 1, T, d))
    Ks = np.empty((L, T, Hkv * hd))
    Vs = np.empty((L, T, Hkv * hd))
    H[0] = h
    mask = np.triu(np.ones((T, T), dtype=bool), k=1)
    for l in range(L):
        a = _rms(h, bf16_to_f64(w["attn_norm"][l]), eps)
        q = (a @ bf16_to_f64(w["wq"][l]).T).reshape(T, Hq, hd)
        k = (a @ bf16_to_f64(w["wk"][l]).T).reshape(T, Hkv, hd)
        v = (a @ bf16_to_f64(w["wv"][l]).T).reshape(T, Hkv, hd)
        q, k = _rope(q, base), _rope(k, base)
        Ks[l], Vs[l] = k.reshape(T, -1), v.reshape(T, -1)
        o = np.empty((T, Hq, hd))
        for j in range(Hq):
            kv = j // (Hq // Hkv)
            s = q[:, j, :] @ k[:, kv, :].T / np.sqrt(hd)
            s[mask] = -np.inf
            s = np.exp(s - s.max(axis=1, keepdims=True))
            s /= s.sum(axis=1, keepdims=True)
            o[:, j, :] = s @ v[:, kv, :]
        h = h + o.reshape(T, Hq * hd) @ bf16_to_f64(w["wo"][l]).T
        m = _rms(h, bf16_to_f64(w["mlp_norm"][l]), eps)
        g = m @ bf16_to_f64(w["w_gate"][l]).T
        u = m @ bf16_to_f64(w["w_up"][l]).T
        h = h + (g / (1.0 + np.exp(-g)) * u) @ bf16_to_f64(w["w_down"][l]).T
        H[l + 1] = h
    return {"H": H, "K": Ks, "V": Vs}


def head_logits(dims: dict, w: dict, layer: int, h: np.ndarray) -> np.ndarray:
    """g_layer(h): RMSNorm then projection, all Vt+Vs logits."""
    a = _rms(h, bf16_to_f64(w["head_norm"][layer - 1]), dims["rms_eps"])
    return bf16_to_f64(w["head_proj"][layer - 1]) @ a


def scheduled_depth(dims: dict, modality: int, c: int) -> int:
    """Sec. IV-B.1: in-chunk index c runs all L layers iff c mod K == r; text always does
    unless text_exit is set (1: text too; 2: text only, speech always full, Sec. V-E row G10).
    Text positions that follow the schedule may have their own (text_period, text_phase)."""
    L, e = dims["n_layers"], dims["exit_layer"]
    te = dims.get("text_exit", 0)
    if (modality == 0 and te == 0) or (modality == 1 and te == 2):
        return L
    K, r = dims["refresh_period"], dims["refresh_phase"]
    if modality == 0 and dims.get("text_period", 0) > 0:      # text positions with a period of their own
        K, r = dims["text_period"], dims.get("text_phase", 0)
    return L if c % K == r else e


def entropy(z: np.ndarray) -> float:
    """Entropy (nats) of softmax(z) (Sec. V-B: the confidence signal of the compared method)."""
    lp = z - z.max()
    lp = lp - np.log(np.exp(lp).sum())
    p = np.exp(lp)
    return float(-(p[p > 0] * lp[p > 0]).sum())


def decode_stream(dims: dict, w: dict, prompt, modalities, counters, forced=None, depths=None):
    """Greedy SPAR-K generation by full recomputation.  `prompt` is the whole prompt (the last
    prompt token is the first step's input).  If `forced` is given its tokens are fed back
    instead of the computed ones (teacher forcing).  Returns a list of per-step dicts.

    The depth of a step is `depths[s]` if given; else, for a modality in dims["conf_modalities"]
    (bit 0 text, bit 1 speech), the first layer l >= conf_start whose head's prediction over the
    modality's ids has entropy < conf_threshold (L if none; Sec. V-B); else the schedule's."""
    toks = list(np.asarray(prompt))
    Vt = dims["vocab_text"]
    V = Vt + dims["vocab_speech"]
    out = []
    for s, (mod, c) in enumerate(zip(modalities, counters)):
        fw = forward_all(dims, w, toks)
        p = len(toks) - 1
        lo, hi = (0, Vt) if mod == 0 else (Vt, V)
        ents = {}
        if depths is not None:
            dep = int(depths[s])
        elif (dims.get("conf_modalities", 0) >> (1 if mod else 0)) & 1:
            dep = dims["n_layers"]
            for l in range(dims["conf_start"], dims["n_layers"]):
                ents[l] = entropy(head_logits(dims, w, l, fw["H"][l, p])[lo:hi])
                if ents[l] < dims["conf_threshold"]:
                    dep = l
                    break
        else:
            dep = scheduled_depth(dims, int(mod), int(c))
        hid = fw["H"][dep, p]
        z = head_logits(dims, w, dep, hid)
        y = lo + int(np.argmax(z[lo:hi]))
        zs = np.sort(z[lo:hi])
        out.append({"token": y, "depth": dep, "hidden": hid, "logits": z, "pos": p,
                    "margin": float(zs[-1] - zs[-2]), "entropies": ents})
        toks.append(int(forced[s]) if forced is not None else y)
    return out

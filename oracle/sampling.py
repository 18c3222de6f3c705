"""Nucleus (top-p) sampling with temperature over a modality's id range (NumPy, float64).

TEST INFRASTRUCTURE: a plain restatement of the decoding rule the paper uses for its 28-layer
backbone (Sec. V-A: nucleus sampling, temperature 0.7, top_p 0.9), independent of the CUDA path.

Definition (Holtzman et al., "The Curious Case of Neural Text Degeneration", the rule the cited
generation configuration names): with p_i = softmax(z_i / T) over the allowed ids, order the ids by
decreasing p_i (equal p: lower id first), keep the shortest prefix whose probability mass reaches
top_p, renormalise, and draw from it.  The draw is made reproducible by passing the uniform number
u in [0, 1) in: the token is the first one in that order whose cumulative mass exceeds u times the
kept mass.
"""
from __future__ import annotations

import numpy as np


def nucleus_order(logits: np.ndarray, lo: int, hi: int, temperature: float):
    """ids of [lo, hi) by decreasing probability (ties: lower id first) and their probabilities."""
    z = np.asarray(logits, dtype=np.float64)[lo:hi] / float(temperature)
    w = np.exp(z - z.max())
    p = w / w.sum()
    order = np.lexsort((np.arange(lo, hi), -p))  # primary key -p, then id
    return order + lo, p[order]


def nucleus_sample(logits: np.ndarray, lo: int, hi: int, temperature: float, top_p: float, u: float) -> dict:
    """Token drawn with the uniform number u; also where u landed, for tolerance-aware checks:
    `ids`/`cum` are the kept ids in order and their cumulative mass divided by the kept mass."""
    ids, p = nucleus_order(logits, lo, hi, temperature)
    cum = np.cumsum(p)
    n_keep = int(np.searchsorted(cum, top_p, side="left")) + 1  # first prefix with mass >= top_p
    n_keep = min(n_keep, len(ids))
    kept = cum[:n_keep] / cum[n_keep - 1]
    j = int(np.searchsorted(kept, u, side="right"))             # first cumulative mass > u
    j = min(j, n_keep - 1)
    return {"token": int(ids[j]), "rank": j, "n_keep": n_keep, "ids": ids[:n_keep], "cum": kept}


def landing_error(sample: dict, token: int, u: float) -> float:
    """How far u lies outside the cumulative interval the reference order gives `token`
    (0 if inside; infinity if the token is not in the kept set)."""
    where = np.nonzero(sample["ids"] == token)[0]
    if len(where) == 0:
        return float("inf")
    j = int(where[0])
    lo = sample["cum"][j - 1] if j > 0 else 0.0
    hi = sample["cum"][j]
    return float(max(lo - u, u - hi, 0.0))

"""Pins for the exit schedule (Sec. IV-B.1) and the LayerSaving metric (Eq. 4)."""
import os
from fractions import Fraction

import pytest

from oracle import oracle as ora
from paper_2603_09215_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "table2_exit_layers.txt")


def _rows():
    out = []
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            row, L, N, sched, e, avg, sav, tol = line.split()
            out.append((row, int(L), int(N), sched, int(e), float(avg), sav, float(tol)))
    return out


def _kr(sched, N):
    # fixed-layer exit = a period longer than the chunk whose full position is never reached
    return {"even": (2, 0), "odd": (2, 1), "triple": (3, 0), "fixed": (N + 1, N)}[sched]


@pytest.mark.parametrize("row", _rows(), ids=lambda r: r[0])
def test_table2_average_exit_layer(row):
    name, L, N, sched, e, avg, sav, tol = row
    K, r = _kr(sched, N)
    depths = [ora.depth(1, c, K, r, e, L) for c in range(N)]
    mean = sum(depths) / N
    assert abs(mean - avg) <= tol, (name, depths, mean)
    saving = (1 - mean / L) * 100  # Eq. 4
    half_ulp = 0.5 if "." not in sav else 0.05
    assert abs(saving - float(sav)) <= half_ulp + (0.1 if tol > 0.01 else 1e-9), (name, saving)


def test_schedule_patterns_from_the_text():
    L, e = 28, 22
    assert [ora.depth(1, c, 2, 0, e, L) for c in range(6)] == [L, e, L, e, L, e]        # Even
    assert [ora.depth(1, c, 2, 1, e, L) for c in range(6)] == [e, L, e, L, e, L]        # Odd
    assert [ora.depth(1, c, 3, 0, e, L) for c in range(7)] == [L, e, e, L, e, e, L]     # Triple
    # text never leaves early in the main rows; it does when the text schedule is switched on
    assert all(ora.depth(0, c, 2, 0, e, L) == L for c in range(8))
    assert [ora.depth(0, c, 2, 0, e, L, 1) for c in range(4)] == [L, e, L, e]
    # a 4-position chunk has two full and two early positions under all three (Sec. V-C)
    for K, r in ((2, 0), (2, 1), (3, 0)):
        d = [ora.depth(1, c, K, r, e, L) for c in range(4)]
        assert d.count(L) == 2 and d.count(e) == 2


def test_text_only_schedule_row_G10():
    """Sec. V-E row G10: the periodic rule on text tokens only; speech stays at full depth."""
    path = os.path.join(os.path.dirname(__file__), "golden", "table2_text_schedule.txt")
    rows = [l.split() for l in open(path) if l.strip() and not l.startswith("#")]
    assert rows
    for name, L, Nt, Ns, sched, e, avg_t, avg_s, tol in rows:
        L, Nt, Ns, e = int(L), int(Nt), int(Ns), int(e)
        K, r = _kr(sched, Nt)
        text = [ora.depth(0, c, K, r, e, L, 2) for c in range(Nt)]
        speech = [ora.depth(1, c, K, r, e, L, 2) for c in range(Ns)]
        assert abs(sum(text) / Nt - float(avg_t)) <= float(tol), (name, text)
        assert sum(speech) / Ns == float(avg_s), (name, speech)
        # on whole periods the printed value is exact
        whole = [ora.depth(0, c, K, r, e, L, 2) for c in range(K * 6)]
        assert sum(whole) / len(whole) == float(avg_t)
    # the three modes side by side (L = 4, e = 2, Even)
    assert [ora.depth(0, c, 2, 0, 2, 4, 0) for c in range(4)] == [4, 4, 4, 4]
    assert [ora.depth(1, c, 2, 0, 2, 4, 0) for c in range(4)] == [4, 2, 4, 2]
    assert [ora.depth(0, c, 2, 0, 2, 4, 1) for c in range(4)] == [4, 2, 4, 2]
    assert [ora.depth(1, c, 2, 0, 2, 4, 1) for c in range(4)] == [4, 2, 4, 2]
    assert [ora.depth(0, c, 2, 0, 2, 4, 2) for c in range(4)] == [4, 2, 4, 2]
    assert [ora.depth(1, c, 2, 0, 2, 4, 2) for c in range(4)] == [4, 4, 4, 4]


def test_full_count_closed_form_against_enumeration():
    # number of full-depth positions in a chunk of N: floor((N - r + K - 1) / K)
    L, e = 40, 30
    for N in range(1, 65):
        for K in range(1, 17):
            for r in range(K):
                n_full = sum(ora.depth(1, c, K, r, e, L) == L for c in range(N))
                assert n_full == (N - r + K - 1) // K, (N, K, r)


def test_mean_depth_identity_on_whole_periods():
    # mean speech depth = (e (K-1) + L) / K exactly whenever K divides the chunk
    for L, e in ((28, 20), (40, 30), (4, 2)):
        for K in range(1, 9):
            for mult in range(1, 5):
                N = K * mult
                for r in range(K):
                    tot = sum(ora.depth(1, c, K, r, e, L) for c in range(N))
                    assert Fraction(tot, N) == Fraction(e * (K - 1) + L, K)
    # otherwise it differs by at most (L-e)(K-1)/(K N)
    for N in range(1, 40):
        for K in range(1, 9):
            tot = sum(ora.depth(1, c, K, 0, 30, 40) for c in range(N))
            gap = abs(Fraction(tot, N) - Fraction(30 * (K - 1) + 40, K))
            assert gap <= Fraction((40 - 30) * (K - 1), K * N)


def test_per_modality_period_and_phase():
    """Sec. V-E asks for different policies for text and speech.  With a period and phase of its
    own per modality each side keeps the closed forms of Sec. IV-B.1 independently: the number of
    full-depth positions of a chunk is floor((N - r + K - 1) / K) with that modality's (K, r), and
    the mean depth over whole periods is (e (K - 1) + L) / K; the paper's own two-sided row G11
    has speech on Even(36) at 38.00 whatever the text side does."""
    L, e = 40, 36
    for Ks, rs, Kt, rt in ((2, 0, 3, 1), (4, 0, 2, 1), (2, 1, 5, 4), (3, 2, 3, 0)):
        for N in (1, 5, 13, 26):
            sp = [ora.depth_mod(1, c, Ks, rs, Kt, rt, e, L, 1) for c in range(N)]
            tx = [ora.depth_mod(0, c, Ks, rs, Kt, rt, e, L, 1) for c in range(N)]
            assert sum(d == L for d in sp) == (N - rs + Ks - 1) // Ks
            assert sum(d == L for d in tx) == (N - rt + Kt - 1) // Kt
            assert set(sp + tx) <= {e, L}
        for K, r, mod in ((Ks, rs, 1), (Kt, rt, 0)):
            whole = [ora.depth_mod(mod, c, Ks, rs, Kt, rt, e, L, 1) for c in range(K * 4)]
            assert Fraction(sum(whole), len(whole)) == Fraction(e * (K - 1) + L, K)
        # the modes that exempt a modality still do
        assert all(ora.depth_mod(0, c, Ks, rs, Kt, rt, e, L, 0) == L for c in range(12))
        assert all(ora.depth_mod(1, c, Ks, rs, Kt, rt, e, L, 2) == L for c in range(12))
        # with the same pair on both sides it is the one-pair rule
        assert [ora.depth_mod(m, c, Ks, rs, Ks, rs, e, L, 1) for m in (0, 1) for c in range(9)] == \
               [ora.depth(m, c, Ks, rs, e, L, 1) for m in (0, 1) for c in range(9)]
    # row G11's speech side: Even(36) on the 26-position chunk of the 40-layer backbone
    assert sum(ora.depth_mod(1, c, 2, 0, 7, 3, 36, 40, 1) for c in range(26)) / 26 == 38.0


def test_K1_and_e_equal_L_are_full_depth():
    assert all(ora.depth(1, c, 1, 0, 5, 9) == 9 for c in range(20))
    assert all(ora.depth(1, c, 4, 0, 9, 9) == 9 for c in range(20))


@pytest.mark.parametrize("name", ["cfg1_tiny_b1", "cfg2_step_b1", "cfg4_glm_b16"])
def test_workload_depth_sequences(name):
    """The depth log of the phase-aligned workloads, and Eq. 4 on it."""
    wl = synth.WORKLOADS[name]
    L = synth.SHAPES[wl["shape"]]["n_layers"]
    e, K, r = wl["exit_layer"], wl["refresh_period"], wl["refresh_phase"]
    log = []
    for g in range(wl["steps"]):
        m, c = synth.interleave(g, wl["n_text"], wl["n_speech"])
        log.append((m, ora.depth(m, c, K, r, e, L)))
    speech = [d for m, d in log if m == 1]
    text = [d for m, d in log if m == 0]
    assert all(d == L for d in text)
    if name == "cfg1_tiny_b1":
        assert speech[:8] == [4, 2, 2, 4, 4, 2, 2, 4]
        assert len(text) == 32 and speech.count(4) == 32 and speech.count(2) == 32
        assert Fraction(sum(speech), len(speech)) == 3
    if name == "cfg2_step_b1":
        assert speech[:4] == [28, 20, 20, 20]
        assert Fraction(sum(speech[:4 * 200]), 800) == Fraction(20 * 3 + 28, 4)
    if name == "cfg4_glm_b16":
        chunk = speech[:26]
        assert chunk.count(40) == 7 and chunk.count(30) == 19
    saving = (1 - (sum(speech) / len(speech)) / L) * 100
    per_pos = sum((L - d) / L for d in speech) / len(speech) * 100   # second form of Eq. 4
    assert abs(saving - per_pos) < 1e-9


def test_interleave_bookkeeping():
    seq = [synth.interleave(g, 2, 4) for g in range(12)]
    assert seq == [(0, 0), (0, 1), (1, 0), (1, 1), (1, 2), (1, 3)] * 2
    # a phase shifts the cycle, an offset shifts the counter
    assert synth.interleave(0, 1, 4, phase=3, offset=2) == (1, 4)
    # running counters keep counting across chunks
    run = [synth.interleave(g, 1, 2, running=True) for g in range(7)]
    assert run == [(0, 0), (1, 0), (1, 1), (0, 0), (1, 2), (1, 3), (0, 0)]

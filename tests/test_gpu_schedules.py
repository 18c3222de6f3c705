"""GPU parity for the schedule variants of Sec. IV-B.1, V-B and V-E: the library is neutral about
the counters the caller passes, so fixed-layer exit, Odd, a counter that runs across chunks and the
text-side schedules are all the same kernels driven differently."""
import pytest
import torch

from paper_2603_09215_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def util():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from tests import parity_util
    return parity_util


CASES = [
    # text_exit, e, K, r, N_text, N_speech, running, max_pending
    (0, 2, 2, 1, 1, 4, False, 2),     # Odd {e, L, e, L}
    (0, 2, 7, 6, 1, 6, False, 6),     # fixed-layer: no refresh inside a chunk, the text step flushes six rows
    (0, 2, 3, 0, 1, 4, True, 3),      # Triple on a counter that runs across chunks
    (1, 2, 2, 0, 3, 4, False, 2),     # text and speech both Even
    (2, 2, 2, 0, 5, 3, False, 2),     # text only (row G10): speech steps flush pending text rows
    (2, 1, 3, 0, 4, 2, False, 3),     # text only, Triple, exit after the first layer
]


@pytest.mark.parametrize("text_exit,e,K,r,nt,ns,running,maxp", CASES)
def test_schedule_variants(util, text_exit, e, K, r, nt, ns, running, maxp):
    dims = synth.model_dims("tiny", e, K, r, text_exit=text_exit)
    w = synth.make_weights(dims, seed=0)
    prompt = synth.make_prompts(dims, 1, 19, 19, seed=21)[0]
    P = util.Pair(dims, w, 1, 19 + 64, maxp, prefill_rows=16)
    P.prefill([prompt])
    depths, mods, pend_max = [], [], 0
    for g in range(44):
        m, c = synth.interleave(g, nt, ns, running=running)
        _, _, dep = P.step([m], [c])
        depths.append(int(dep[0]))
        mods.append(m)
        pend_max = max(pend_max, P.g.slot_state(0)[1])
    L = dims["n_layers"]
    assert e in depths and L in depths
    if text_exit == 0:
        assert all(d == L for d, m in zip(depths, mods) if m == 0)
    if text_exit == 2:
        assert all(d == L for d, m in zip(depths, mods) if m == 1)
        assert any(d == e for d, m in zip(depths, mods) if m == 0)
    if K > ns and text_exit == 0:    # fixed-layer exit
        assert all(d == e for d, m in zip(depths, mods) if m == 1) and pend_max == ns
    ln, pend = P.g.slot_state(0)
    P.check_cache(0, range(1, e + 1), ln)
    P.check_cache(0, range(e + 1, L + 1), ln - pend)
    assert P.stats["tok_checked"] > 3, P.stats
    P.close()


def test_text_side_schedule_in_a_mixed_batch(util):
    """Five sequences at different interleave phases with the text-only schedule: every step mixes
    early-exit text rows, full-depth text rows and full-depth speech rows that flush pending ones."""
    dims = synth.model_dims("tiny", 2, 2, 0, text_exit=2)
    w = synth.make_weights(dims, seed=0)
    B = 5
    prompts = synth.make_prompts(dims, B, 8, 40, seed=14)
    phi, off = synth.make_phases(B, 4, 3, 2, True, seed=3)
    P = util.Pair(dims, w, B, 40 + 48, 2, prefill_rows=16)
    P.prefill(prompts)
    mixed = 0
    for g in range(36):
        mc = [synth.interleave(g, 4, 3, int(p), 0) for p in phi]
        _, _, dep = P.step([m for m, _ in mc], [c for _, c in mc])
        mixed += len(set(int(x) for x in dep)) > 1
    assert mixed > 10
    for s in range(B):
        ln, pend = P.g.slot_state(s)
        P.check_cache(s, range(1, 3), ln)
        P.check_cache(s, range(3, 5), ln - pend)
    P.close()


@pytest.mark.parametrize("text_exit,K,r,tp,tr,nt,ns,maxp", [
    (1, 4, 0, 3, 1, 6, 8, 5),     # speech Triple-like (K = 4), text with period 3 and phase 1
    (2, 2, 0, 3, 2, 6, 2, 3),     # text only with its own period; speech steps are full depth
])
def test_period_and_phase_per_modality(util, text_exit, K, r, tp, tr, nt, ns, maxp):
    """Sec. V-E: text and speech may need different policies.  Each modality follows the periodic
    rule with its own (period, phase); pending rows of either modality are pushed through the
    upper layers by the next full-depth step of either."""
    dims = synth.model_dims("tiny", 2, K, r, text_exit=text_exit, text_period=tp, text_phase=tr)
    w = synth.make_weights(dims, seed=0)
    B = 3
    prompts = synth.make_prompts(dims, B, 10, 30, seed=17)
    P = util.Pair(dims, w, B, 30 + 64, maxp, prefill_rows=16)
    P.prefill(prompts)
    L, e = dims["n_layers"], dims["exit_layer"]
    phases = [0, 5, 9]
    for g in range(42):
        mc = [synth.interleave(g, nt, ns, ph) for ph in phases]
        mods, ctrs = [m for m, _ in mc], [c for _, c in mc]
        _, _, dep = P.step(mods, ctrs)
        for m, c, d in zip(mods, ctrs, dep):
            if m == 0:
                assert d == (L if c % tp == tr else e)
            else:
                assert d == (L if (text_exit == 2 or c % K == r) else e)
    for s in range(B):
        ln, pend = P.g.slot_state(s)
        P.check_cache(s, range(1, e + 1), ln)
        P.check_cache(s, range(e + 1, L + 1), ln - pend)
    assert P.stats["flushes"] > 5 and P.stats["tok_checked"] > 10, P.stats
    P.close()

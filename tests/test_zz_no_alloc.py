"""The attention entry point for callers that cannot allocate device memory.

Some users of this library run where no allocator can be called: inside another engine's fixed
memory plan, or on a path where cudaMalloc is off limits because it synchronises the device.
sparsk_attention_static serves them from a scratch area built into the library.  This test calls
it through the C ABI, twice in a row on different inputs (the area keeps the first call's
contents), and checks each result against sparsk_attention run with caller-provided scratch and
against the CPU oracle's softmax attention.
It lives in a file that is collected last, and passes both alone and after the other tests.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

REL_TOL = 2e-2   # the tolerance of the attention parity tests


def _case(seed, groups, Hq=28, Hkv=4, hd=128, S=900):
    from tests.test_gpu_attention import make_case
    n_slots = 1 + max(s for s, _, _ in groups)
    q, k, v, row_slot, row_pos, g0, gn = make_case(seed, n_slots, Hq, Hkv, hd, S, groups)
    t = lambda a: torch.tensor(a, dtype=torch.int32, device="cuda")
    keep = dict(q=q.cuda(), k=k.cuda(), v=v.cuda(), rs=t(row_slot), rp=t(row_pos), g0=t(g0), gn=t(gn))
    keep["meta"] = (max(gn), max(row_pos) + 1, Hq, hd)
    return keep


def _run(binding, c, static):
    mg, ml, Hq, hd = c["meta"]
    out = torch.full((c["q"].shape[0], Hq * hd), float("nan"), dtype=torch.bfloat16, device="cuda")
    args = binding.attn_args(c["q"], c["k"], c["v"], out, c["rs"], c["rp"], c["g0"], c["gn"], mg, ml, Hq)
    if static:
        rc, msg = binding.attention_static(args)
        assert rc == binding.OK, msg
    else:
        scratch = torch.empty(binding.attention_scratch_bytes(c["q"].shape[0], Hq, hd), dtype=torch.uint8,
                              device="cuda")
        assert binding.attention(args, scratch) == binding.OK
    torch.cuda.synchronize()
    return out.float().cpu().numpy()


def test_static_scratch_attention_matches_the_allocating_entry_point():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2603_09215_b200 import binding
    first = _case(11, [(0, 700, 4), (1, 64, 1), (2, 333, 2)])
    second = _case(12, [(1, 10, 1), (0, 850, 3)])            # fewer rows, other lengths: stale cells remain
    from tests.test_gpu_attention import oracle_out
    for c in (first, second):
        ref = _run(binding, c, static=False)
        got = _run(binding, c, static=True)
        assert np.isfinite(got).all()
        err = np.abs(got - ref).max() / np.abs(ref).max()
        assert err <= REL_TOL, err
        # and directly against the CPU oracle's softmax attention, row by row and head by head
        _, _, Hq, hd = c["meta"]
        want = oracle_out(c["q"].cpu(), c["k"].cpu(), c["v"].cpu(), c["rs"].cpu().tolist(), c["rp"].cpu().tolist(),
                          Hq, c["k"].shape[1], hd)
        err = np.abs(got - want).max() / np.abs(want).max()
        assert err <= REL_TOL, err
    # a call whose partials do not fit the built-in area is refused, with the sizes in the message
    big = _case(13, [(0, 0, 1)], Hq=32, Hkv=2, hd=128, S=8)
    mg, ml, Hq, hd = big["meta"]
    n_rows = 1024
    out = torch.zeros((n_rows, Hq * hd), dtype=torch.bfloat16, device="cuda")
    args = binding.attn_args(big["q"], big["k"], big["v"], out, big["rs"], big["rp"], big["g0"], big["gn"],
                             mg, ml, Hq)
    args.n_rows = n_rows
    assert binding.attention_scratch_bytes(n_rows, Hq, hd) > binding.STATIC_SCRATCH_BYTES
    rc, msg = binding.attention_static(args)
    assert rc == binding.ECAPACITY and str(binding.STATIC_SCRATCH_BYTES) in msg, (rc, msg)

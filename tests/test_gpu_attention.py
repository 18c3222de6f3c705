"""Per-kernel parity: the stand-alone split-KV attention entry point against the oracle's
single-head softmax attention, on ragged groups that span several tiles and splits."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

REL_TOL = 2e-2


def make_case(seed, n_slots, Hq, Hkv, hd, S, groups):
    """groups: list of (slot, pos0, nrows).  Queries rounded to bf16, keys and values to fp16."""
    g = torch.Generator("cpu").manual_seed(seed)
    n_rows = sum(n for _, _, n in groups)
    q = torch.randn((n_rows, Hq * hd), generator=g).to(torch.bfloat16)
    k = torch.randn((n_slots, Hkv, S, hd), generator=g).to(torch.float16)    # the cache's element type
    v = torch.randn((n_slots, Hkv, S, hd), generator=g).to(torch.float16)
    row_slot, row_pos, g0, gn = [], [], [], []
    for slot, pos0, n in groups:
        g0.append(len(row_slot)); gn.append(n)
        for r in range(n):
            row_slot.append(slot); row_pos.append(pos0 + r)
    return q, k, v, row_slot, row_pos, g0, gn


def oracle_out(q, k, v, row_slot, row_pos, Hq, Hkv, hd):
    from oracle import oracle as ora
    qf, kf, vf = q.double().numpy(), k.double().numpy(), v.double().numpy()
    G = Hq // Hkv
    out = np.zeros_like(qf)
    for i, (s, p) in enumerate(zip(row_slot, row_pos)):
        for j in range(Hq):
            o, _ = ora.attend(qf[i, j * hd:(j + 1) * hd], kf[s, j // G, :p + 1], vf[s, j // G, :p + 1])
            out[i, j * hd:(j + 1) * hd] = o
    return out


@pytest.mark.parametrize("Hq,Hkv,hd,S,groups", [
    (4, 2, 64, 300, [(0, 0, 1), (1, 31, 1), (0, 32, 1), (1, 255, 3)]),          # length 1, tile edges
    (7, 1, 128, 1200, [(0, 1100, 4), (1, 17, 1), (2, 640, 2)]),                  # 7 q heads per kv head
    (32, 2, 128, 700, [(1, 600, 4), (0, 3, 2)]),                                 # 16 per kv head: 2 q blocks
    (6, 2, 64, 400, [(0, 100, 40)]),                                             # prefill-like block of 40 rows
    (8, 2, 128, 500, [(0, 14, 2), (1, 15, 2), (2, 16, 2), (0, 400, 1), (1, 47, 2)]),  # two rows = 8 query vectors: the transposed form, masks at tile edges
])
def test_attention_matches_oracle(Hq, Hkv, hd, S, groups):
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2603_09215_b200 import binding
    n_slots = 1 + max(s for s, _, _ in groups)
    q, k, v, row_slot, row_pos, g0, gn = make_case(3, n_slots, Hq, Hkv, hd, S, groups)
    dev = "cuda"
    t = lambda a: torch.tensor(a, dtype=torch.int32, device=dev)
    out = torch.full((q.shape[0], Hq * hd), float("nan"), dtype=torch.bfloat16, device=dev)
    qd, kd, vd = q.to(dev), k.to(dev), v.to(dev)
    rs, rp, tg0, tgn = t(row_slot), t(row_pos), t(g0), t(gn)
    args = binding.attn_args(qd, kd, vd, out, rs, rp, tg0, tgn, max(gn), max(row_pos) + 1, Hq)
    scratch = torch.empty(binding.attention_scratch_bytes(q.shape[0], Hq, hd), dtype=torch.uint8, device=dev)
    assert binding.attention(args, scratch) == binding.OK
    torch.cuda.synchronize()
    ref = oracle_out(q, k, v, row_slot, row_pos, Hq, Hkv, hd)
    got = out.float().cpu().double().numpy()
    assert np.isfinite(got).all()
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err <= REL_TOL, err


def test_attention_rejects_bad_arguments():
    if not torch.cuda.is_available():
        pytest.skip("needs a CUDA device")
    from paper_2603_09215_b200 import binding
    q, k, v, row_slot, row_pos, g0, gn = make_case(1, 1, 4, 2, 64, 64, [(0, 5, 1)])
    dev = "cuda"
    t = lambda a: torch.tensor(a, dtype=torch.int32, device=dev)
    out = torch.zeros((1, 256), dtype=torch.bfloat16, device=dev)
    keep = [q.to(dev), k.to(dev), v.to(dev), t(row_slot), t(row_pos), t(g0), t(gn)]   # stay alive
    args = binding.attn_args(keep[0], keep[1], keep[2], out, keep[3], keep[4], keep[5], keep[6], 1, 6, 4)
    scratch = torch.empty(binding.attention_scratch_bytes(1, 4, 64), dtype=torch.uint8, device=dev)
    assert binding.attention(args, scratch[:1024]) == binding.EINVAL        # scratch too small
    args.head_dim = 96
    assert binding.attention(args, scratch) == binding.EINVAL
    args.head_dim = 64
    args.max_len = 65                                                        # beyond the cache
    assert binding.attention(args, scratch) == binding.EINVAL
    # a row that names a slot outside the cache reads nothing and yields zeros
    args.max_len = 6
    bad = t([7])
    args.row_slot = bad.data_ptr()
    assert binding.attention(args, scratch) == binding.OK
    torch.cuda.synchronize()
    assert float(out.abs().max()) == 0.0

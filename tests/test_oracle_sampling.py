"""Pins for the reference nucleus sampler (Sec. V-A: temperature 0.7, top_p 0.9 for the 28-layer
backbone): a worked example by hand, limits that reduce to arg max, the inverse-CDF property, the
id range restriction and the tie order."""
import numpy as np

from oracle import sampling as smp


def test_worked_example_by_hand():
    z = np.log(np.array([0.05, 0.5, 0.15, 0.3]))          # ids 0..3; p = those values at T = 1
    s = smp.nucleus_sample(z, 0, 4, 1.0, 0.9, 0.5)
    # order 1 (0.5), 3 (0.3), 2 (0.15), 0 (0.05); cumulative 0.5, 0.8, 0.95: three ids reach 0.9
    assert list(s["ids"]) == [1, 3, 2] and s["n_keep"] == 3
    np.testing.assert_allclose(s["cum"], np.array([0.5, 0.8, 0.95]) / 0.95, rtol=1e-12)
    assert s["token"] == 1                                 # 0.5 < 0.5 / 0.95
    assert smp.nucleus_sample(z, 0, 4, 1.0, 0.9, 0.6)["token"] == 3
    assert smp.nucleus_sample(z, 0, 4, 1.0, 0.9, 0.9)["token"] == 2
    assert smp.nucleus_sample(z, 0, 4, 1.0, 0.9, 0.999999)["token"] == 2   # id 0 is cut off
    # temperature 0.5 squares the probabilities: 0.25, 0.09, 0.0225, 0.0025 (sum 0.365)
    s = smp.nucleus_sample(z, 0, 4, 0.5, 0.9, 0.7)
    np.testing.assert_allclose(s["cum"][0], (0.25 / 0.365) / ((0.25 + 0.09) / 0.365), rtol=1e-12)
    assert s["n_keep"] == 2 and s["token"] == 1 and smp.nucleus_sample(z, 0, 4, 0.5, 0.9, 0.8)["token"] == 3
    # mass reached exactly: top_p = 0.8 keeps two ids, not three
    assert smp.nucleus_sample(np.log(np.array([0.5, 0.25, 0.25])), 0, 3, 1.0, 0.75, 0.0)["n_keep"] == 2


def test_limits_reduce_to_argmax():
    g = np.random.Generator(np.random.PCG64(4))
    z = g.normal(0, 1.0, 300)
    for u in (0.0, 0.3, 0.999):
        assert smp.nucleus_sample(z, 0, 300, 0.7, 1e-12, u)["token"] == int(np.argmax(z))
        assert smp.nucleus_sample(z, 0, 300, 1e-4, 0.9, u)["token"] == int(np.argmax(z))
        assert smp.nucleus_sample(z, 100, 200, 0.7, 1e-12, u)["token"] == 100 + int(np.argmax(z[100:200]))


def test_inverse_cdf_property_and_cutoff():
    """With u on a regular grid every kept id is drawn in proportion to its renormalised softmax
    probability (to within one grid cell), and ids outside the nucleus are never drawn."""
    g = np.random.Generator(np.random.PCG64(5))
    z = g.normal(0, 2.0, 40)
    T, top_p, N = 0.7, 0.9, 20000
    p = np.exp(z / T - np.max(z / T)); p /= p.sum()
    order = np.argsort(-p, kind="stable")
    n_keep = int(np.argmax(np.cumsum(p[order]) >= top_p)) + 1
    kept = order[:n_keep]
    counts = np.zeros(40, int)
    for k in range(N):
        counts[smp.nucleus_sample(z, 0, 40, T, top_p, (k + 0.5) / N)["token"]] += 1
    assert counts.sum() == N and set(np.nonzero(counts)[0]) == set(kept.tolist())
    np.testing.assert_allclose(counts[kept] / N, p[kept] / p[kept].sum(), atol=1.5 / N)
    # the kept mass reaches top_p and would not without its last id
    assert p[kept].sum() >= top_p > p[kept[:-1]].sum()


def test_ties_go_to_the_lower_id_and_range_is_respected():
    z = np.zeros(10)
    s = smp.nucleus_sample(z, 2, 8, 0.7, 1.0, 0.0)
    assert list(s["ids"]) == [2, 3, 4, 5, 6, 7]
    assert [smp.nucleus_sample(z, 2, 8, 0.7, 1.0, u)["token"] for u in (0.0, 0.17, 0.55, 0.99)] == [2, 3, 5, 7]
    # landing_error: zero inside the token's interval, the distance outside, inf outside the kept set
    s = smp.nucleus_sample(z, 2, 8, 0.7, 1.0, 0.55)
    assert smp.landing_error(s, 5, 0.55) == 0.0
    assert abs(smp.landing_error(s, 2, 0.55) - (0.55 - 1 / 6)) < 1e-12
    assert abs(smp.landing_error(s, 7, 0.55) - (5 / 6 - 0.55)) < 1e-12
    assert smp.landing_error(s, 9, 0.55) == float("inf")

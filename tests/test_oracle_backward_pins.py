"""Pins of the oracle's backward pass against something other than itself: central finite differences of
the oracle's FORWARD pass (a different routine), closed-form special cases, and invariants."""
import numpy as np
import pytest

from oracle import agent_attention_oracle as orc


def _problem(seed, B=2, heads=2, H=4, W=6, d=5, pool=(2, 3), bias=True, dwc=True):
    rng = np.random.default_rng(seed)
    N, n = H * W, pool[0] * pool[1]
    p = dict(q=rng.normal(size=(B, heads, N, d)), k=rng.normal(size=(B, heads, N, d)), v=rng.normal(size=(B, heads, N, d)),
             b1=rng.normal(size=(heads, n, N)) * 0.5 if bias else None,
             b2=rng.normal(size=(heads, N, n)) * 0.5 if bias else None,
             wd=rng.normal(size=(heads, d, 3, 3)) * 0.3 if dwc else None,
             g=rng.normal(size=(B, heads, N, d)), H=H, W=W, pool=pool)
    return p


def _loss(p, **over):
    a = {**p, **over}
    o = orc.forward(a["q"], a["k"], a["v"], a["H"], a["W"], pool_hw=a["pool"], b1=a["b1"], b2=a["b2"],
                    dwc_weight=a["wd"], scale1=a.get("s1"), scale2=a.get("s2"))
    return float((o * a["g"]).sum())


def _fd(p, name, idx, eps=1e-5):
    x = p[name].copy()
    x[idx] += eps
    up = _loss(p, **{name: x})
    x[idx] -= 2 * eps
    dn = _loss(p, **{name: x})
    return (up - dn) / (2 * eps)


@pytest.mark.parametrize("seed,kw", [(0, {}), (1, dict(H=6, W=6, pool=(3, 3), d=4)), (2, dict(bias=False, dwc=False)),
                                    (3, dict(H=5, W=7, pool=(2, 2), heads=1))])
def test_backward_matches_finite_differences_of_the_forward_pass(seed, kw):
    p = _problem(seed, **kw)
    p["s1"], p["s2"] = 0.7, 0.4                               # distinct scales: a swap would show
    gr = orc.backward(p["q"], p["k"], p["v"], p["g"], p["H"], p["W"], p["pool"], b1=p["b1"], b2=p["b2"],
                      dwc_weight=p["wd"], scale1=p["s1"], scale2=p["s2"])
    rng = np.random.default_rng(100 + seed)
    pairs = [("q", "dq"), ("k", "dk"), ("v", "dv")]
    if p["b1"] is not None: pairs += [("b1", "db1"), ("b2", "db2")]
    if p["wd"] is not None: pairs += [("wd", "dwd")]
    for name, gname in pairs:
        for _ in range(12):
            idx = tuple(int(rng.integers(0, s)) for s in p[name].shape)
            fd = _fd(p, name, idx)
            assert abs(fd - gr[gname][idx]) <= 1e-6 * max(1.0, abs(fd)), (name, idx, fd, gr[gname][idx])


def test_value_gradient_is_linear_map_transposed():
    # O is linear in V: <dO, O(V)> = <dV, V> exactly (adjoint identity), for any V
    p = _problem(7)
    gr = orc.backward(p["q"], p["k"], p["v"], p["g"], p["H"], p["W"], p["pool"], b1=p["b1"], b2=p["b2"], dwc_weight=p["wd"])
    assert np.isclose(_loss(p), float((gr["dv"] * p["v"]).sum()), rtol=1e-10)


def test_bias_gradients_sum_to_zero_along_the_softmax_axis():
    # a softmax is invariant to a shift of its logits: the gradient with respect to them sums to zero per row
    p = _problem(8)
    gr = orc.backward(p["q"], p["k"], p["v"], p["g"], p["H"], p["W"], p["pool"], b1=p["b1"], b2=p["b2"], dwc_weight=p["wd"])
    assert np.abs(gr["db1"].sum(axis=2)).max() < 1e-10        # rows of B1 run over tokens
    assert np.abs(gr["db2"].sum(axis=2)).max() < 1e-10        # rows of B2 run over agents


def test_uniform_attention_closed_form():
    # zero Q and K and no bias: both softmaxes are uniform, O = mean(V) + DWC(V), so without DWC
    # dV[j] = (1/N) sum_i dO[i] for every token j, and dQ = dK = 0 ... up to the pooling path, also 0
    p = _problem(9, bias=False, dwc=False)
    p["q"][:] = 0.0
    p["k"][:] = 0.0
    gr = orc.backward(p["q"], p["k"], p["v"], p["g"], p["H"], p["W"], p["pool"])
    expect = np.broadcast_to(p["g"].mean(axis=2, keepdims=True), p["g"].shape)
    assert np.allclose(gr["dv"], expect, atol=1e-12)
    assert np.abs(gr["dk"]).max() < 1e-12

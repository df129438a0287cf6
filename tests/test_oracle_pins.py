"""Pins of the fp64 oracle against what the paper and the mathematics fix.

The paper prints no worked numeric example of the operator, so the pins are identities
(Eq. 4), closed forms, special cases that reduce to library routines (each stage is a
conventional Softmax attention, Eq. 3; pooling; a depthwise convolution) and the
hand-evaluated cost model of Eq. 7.  None of these tests touches the CUDA library.
"""
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import agent_attention_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rng(seed):
    return np.random.default_rng(seed)


def _slab(seed, H, W, d, scale=1.0):
    r = _rng(seed)
    N = H * W
    return (r.standard_normal((N, d)) * scale, r.standard_normal((N, d)) * scale,
            r.standard_normal((N, d)))


# ----------------------------------------------------------------------------- Eq. 4
@pytest.mark.parametrize("with_bias", [False, True])
def test_eq4_explicit_matrix_is_row_stochastic_and_matches_two_stage(with_bias):
    H, W, d, ph, pw = 3, 4, 5, 2, 2
    N, n = H * W, ph * pw
    q, k, v = _slab(1, H, W, d)
    a = orc.pool(q, H, W, ph, pw)
    r = _rng(2)
    b1 = r.standard_normal((n, N)) if with_bias else None
    b2 = r.standard_normal((N, n)) if with_bias else None
    m, o_explicit = orc.explicit(q, a, k, v, b1, b2)
    assert m.shape == (N, N)
    assert np.all(m >= 0.0)
    np.testing.assert_allclose(m.sum(axis=1), np.ones(N), atol=1e-12)
    o = orc.forward(q[None, None], k[None, None], v[None, None], H, W, pool_hw=(ph, pw),
                    b1=None if b1 is None else b1[None], b2=None if b2 is None else b2[None])
    np.testing.assert_allclose(o[0, 0], o_explicit, atol=1e-12)
    # and the explicit product written out independently with numpy
    def sm(x):
        e = np.exp(x - x.max(axis=1, keepdims=True))
        return e / e.sum(axis=1, keepdims=True)
    s = d ** -0.5
    phi_q = sm(q @ a.T * s + (0 if b2 is None else b2))
    phi_k = sm(a @ k.T * s + (0 if b1 is None else b1))
    np.testing.assert_allclose(m, phi_q @ phi_k, atol=1e-12)
    np.testing.assert_allclose(o[0, 0], phi_q @ (phi_k @ v), atol=1e-12)


# ------------------------------------------------------------------ spec checks
def test_single_agent_gives_identical_rows():
    H, W, d = 4, 5, 6
    q, k, v = _slab(3, H, W, d)
    o, a, va = orc.forward(q[None, None], k[None, None], v[None, None], H, W,
                           pool_hw=(1, 1), return_intermediates=True)
    np.testing.assert_allclose(a[0, 0, 0], q.mean(axis=0), atol=1e-14)
    for i in range(H * W):
        np.testing.assert_allclose(o[0, 0, i], va[0, 0, 0], atol=1e-14)


@pytest.mark.parametrize("with_bias", [False, True])
def test_constant_v_is_reproduced(with_bias):
    H, W, d, p = 6, 6, 4, 3
    N, n = H * W, p * p
    q, k, _ = _slab(4, H, W, d)
    const = np.array([0.5, -2.0, 3.25, 7.0])
    v = np.tile(const, (N, 1))
    r = _rng(5)
    b1 = r.standard_normal((1, n, N)) if with_bias else None
    b2 = r.standard_normal((1, N, n)) if with_bias else None
    o = orc.forward(q[None, None], k[None, None], v[None, None], H, W, pool_hw=(p, p),
                    b1=b1, b2=b2)
    np.testing.assert_allclose(o[0, 0], v, atol=1e-12)


def test_key_value_permutation_invariance():
    H, W, d, p = 6, 4, 8, 2
    N = H * W
    q, k, v = _slab(6, H, W, d)
    perm = _rng(7).permutation(N)
    o1, _, va1 = orc.forward(q[None, None], k[None, None], v[None, None], H, W,
                             pool_hw=(p, p), return_intermediates=True)
    o2, _, va2 = orc.forward(q[None, None], k[perm][None, None], v[perm][None, None], H, W,
                             pool_hw=(p, p), return_intermediates=True)
    np.testing.assert_allclose(va1, va2, atol=1e-12)
    np.testing.assert_allclose(o1, o2, atol=1e-12)


# ------------------------------------------------ each stage = library Softmax attention
def test_each_stage_equals_library_sdpa_with_additive_mask():
    B, heads, H, W, d, p = 2, 3, 6, 8, 16, 3
    N, n = H * W, p * p
    r = _rng(8)
    q = r.standard_normal((B, heads, N, d))
    k = r.standard_normal((B, heads, N, d))
    v = r.standard_normal((B, heads, N, d))
    b1 = r.standard_normal((heads, n, N))
    b2 = r.standard_normal((heads, N, n))
    s1, s2 = 0.31, 0.47                         # distinct, so a swapped scale shows
    o, a, va = orc.forward(q, k, v, H, W, pool_hw=(p, p), b1=b1, b2=b2,
                           scale1=s1, scale2=s2, return_intermediates=True, threads=2)
    tq, tk, tv = (torch.from_numpy(x) for x in (q, k, v))
    ta = F.adaptive_avg_pool2d(
        tq.reshape(B * heads, H, W, d).permute(0, 3, 1, 2).contiguous(), (p, p))
    ta = ta.reshape(B, heads, d, n).transpose(-1, -2).contiguous()
    np.testing.assert_allclose(a, ta.numpy(), atol=1e-13)
    tva = F.scaled_dot_product_attention(ta, tk, tv, attn_mask=torch.from_numpy(b1)[None],
                                         scale=s1)
    np.testing.assert_allclose(va, tva.numpy(), atol=1e-12)
    to = F.scaled_dot_product_attention(tq, ta, tva, attn_mask=torch.from_numpy(b2)[None],
                                        scale=s2)
    np.testing.assert_allclose(o, to.numpy(), atol=1e-12)


def test_default_scale_is_inverse_sqrt_d():
    H, W, d = 4, 4, 9
    q, k, v = _slab(9, H, W, d)
    o = orc.forward(q[None, None], k[None, None], v[None, None], H, W, pool_hw=(2, 2))
    o_explicit = orc.forward(q[None, None], k[None, None], v[None, None], H, W, pool_hw=(2, 2),
                             scale1=1.0 / 3.0, scale2=1.0 / 3.0)
    np.testing.assert_allclose(o, o_explicit, atol=1e-14)


def test_user_agents_equal_queries_reduces_to_nested_softmax_attention():
    H, W, d = 3, 3, 4
    q, k, v = _slab(10, H, W, d)
    o = orc.forward(q[None, None], k[None, None], v[None, None], H, W, agents=q[None, None])
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (q, k, v))
    inner = F.scaled_dot_product_attention(tq, tk, tv)
    outer = F.scaled_dot_product_attention(tq, tq, inner)
    np.testing.assert_allclose(o, outer.numpy(), atol=1e-12)


# ------------------------------------------------------------------------------ pooling
@pytest.mark.parametrize("H,W,ph,pw", [(14, 14, 7, 7), (10, 10, 4, 4), (7, 9, 3, 2),
                                       (5, 5, 5, 5), (6, 6, 1, 1), (11, 13, 4, 5)])
def test_pool_equals_library_adaptive_avg_pool(H, W, ph, pw):
    d = 3
    q = _rng(11).standard_normal((H * W, d))
    a = orc.pool(q, H, W, ph, pw)
    t = torch.from_numpy(q).reshape(H, W, d).permute(2, 0, 1)[None]
    ref = F.adaptive_avg_pool2d(t, (ph, pw))[0].reshape(d, ph * pw).T
    np.testing.assert_allclose(a, ref.numpy(), atol=1e-14)


def test_pool_closed_forms():
    H, W, d = 6, 8, 2
    const = np.tile(np.array([1.5, -4.0]), (H * W, 1))
    np.testing.assert_allclose(orc.pool(const, H, W, 3, 4), np.tile([1.5, -4.0], (12, 1)),
                               atol=1e-15)
    q = _rng(12).standard_normal((H * W, d))
    np.testing.assert_allclose(orc.pool(q, H, W, 1, 1)[0], q.mean(axis=0), atol=1e-15)
    np.testing.assert_allclose(orc.pool(q, H, W, H, W), q, atol=0)
    # block averaging when the pool divides the grid: agent (1,2) of a 3x4 pool = rows 2..3, cols 4..5
    blk = q.reshape(H, W, d)[2:4, 4:6].reshape(-1, d).mean(axis=0)
    np.testing.assert_allclose(orc.pool(q, H, W, 3, 4)[1 * 4 + 2], blk, atol=1e-15)


# ---------------------------------------------------------------------------------- DWC
def test_dwc_equals_library_depthwise_conv():
    H, W, d = 7, 5, 6
    r = _rng(13)
    v = r.standard_normal((H * W, d))
    wd = r.standard_normal((d, 3, 3))
    got = orc.dwc(v, wd, H, W)
    t = torch.from_numpy(v).reshape(H, W, d).permute(2, 0, 1)[None]
    ref = F.conv2d(t, torch.from_numpy(wd)[:, None], padding=1, groups=d)[0]
    np.testing.assert_allclose(got, ref.permute(1, 2, 0).reshape(H * W, d).numpy(), atol=1e-13)


def test_dwc_centre_tap_is_the_stable_diffusion_shortcut():
    # App. C.1: O = ... + kV is the module with a filter that is k at the centre, 0 elsewhere.
    H, W, d, kk = 4, 6, 3, 0.075
    v = _rng(14).standard_normal((H * W, d))
    wd = np.zeros((d, 3, 3))
    wd[:, 1, 1] = kk
    np.testing.assert_allclose(orc.dwc(v, wd, H, W), kk * v, atol=1e-16)


def test_dwc_corner_tap_shifts_without_flip_and_pads_with_zero():
    H, W, d = 4, 5, 2
    v = _rng(15).standard_normal((H * W, d))
    wd = np.zeros((d, 3, 3))
    wd[:, 0, 0] = 1.0                      # tap (u=0, v=0) reads V[y-1, x-1]
    got = orc.dwc(v, wd, H, W).reshape(H, W, d)
    vv = v.reshape(H, W, d)
    np.testing.assert_allclose(got[1:, 1:], vv[:-1, :-1], atol=0)
    assert np.all(got[0] == 0) and np.all(got[:, 0] == 0)
    wd[:] = 0
    wd[:, 2, 1] = 1.0                      # tap (u=2, v=1) reads V[y+1, x]
    got = orc.dwc(v, wd, H, W).reshape(H, W, d)
    np.testing.assert_allclose(got[:-1], vv[1:], atol=0)
    assert np.all(got[-1] == 0)


def test_dwc_is_per_head_and_added_to_attention_term():
    B, heads, H, W, d, p = 2, 2, 4, 4, 3, 2
    r = _rng(16)
    q, k, v = (r.standard_normal((B, heads, H * W, d)) for _ in range(3))
    wd = r.standard_normal((heads, d, 3, 3))
    o_att = orc.forward(q, k, v, H, W, pool_hw=(p, p))
    o = orc.forward(q, k, v, H, W, pool_hw=(p, p), dwc_weight=wd)
    for b in range(B):
        for h in range(heads):
            np.testing.assert_allclose(o[b, h] - o_att[b, h], orc.dwc(v[b, h], wd[h], H, W),
                                       atol=1e-13)


# --------------------------------------------------------------------------- closed forms
def test_zero_queries_give_the_mean_of_v():
    H, W, d, p = 5, 4, 3, 2
    _, k, v = _slab(17, H, W, d)
    q = np.zeros_like(k)
    o = orc.forward(q[None, None], k[None, None], v[None, None], H, W, pool_hw=(p, p))
    np.testing.assert_allclose(o[0, 0], np.tile(v.mean(axis=0), (H * W, 1)), atol=1e-13)


def test_bias_shift_invariance_and_one_hot_limit():
    H, W, d, p = 4, 4, 5, 2
    N, n = H * W, p * p
    q, k, v = _slab(18, H, W, d)
    r = _rng(19)
    b1 = r.standard_normal((1, n, N))
    b2 = r.standard_normal((1, N, n))
    args = (q[None, None], k[None, None], v[None, None], H, W)
    o = orc.forward(*args, pool_hw=(p, p), b1=b1, b2=b2)
    b1s = b1 + r.standard_normal((1, n, 1))       # a constant per agent row of B1
    b2s = b2 + r.standard_normal((1, N, 1))       # a constant per query row of B2
    np.testing.assert_allclose(orc.forward(*args, pool_hw=(p, p), b1=b1s, b2=b2s), o, atol=1e-12)
    # B1 that leaves one key per agent: V_A[a] is that key's value row
    pick = r.integers(0, N, size=n)
    hard = np.full((1, n, N), -1e9)
    hard[0, np.arange(n), pick] = 0.0
    _, _, va = orc.forward(*args, pool_hw=(p, p), b1=hard, return_intermediates=True)
    np.testing.assert_allclose(va[0, 0], v[pick], atol=1e-12)
    # B2 that leaves one agent per query: O[i] = V_A[that agent]
    pick2 = r.integers(0, n, size=N)
    hard2 = np.full((1, N, n), -1e9)
    hard2[0, np.arange(N), pick2] = 0.0
    o2, _, va2 = orc.forward(*args, pool_hw=(p, p), b2=hard2, return_intermediates=True)
    np.testing.assert_allclose(o2[0, 0], va2[0, 0][pick2], atol=1e-12)


def test_bias_is_indexed_per_head_and_shared_over_batch():
    B, heads, H, W, d, p = 2, 3, 3, 4, 4, 2
    N, n = H * W, p * p
    r = _rng(20)
    q, k, v = (r.standard_normal((B, heads, N, d)) for _ in range(3))
    b1 = r.standard_normal((heads, n, N))
    b2 = r.standard_normal((heads, N, n))
    o = orc.forward(q, k, v, H, W, pool_hw=(p, p), b1=b1, b2=b2, threads=3)
    for b in range(B):
        for h in range(heads):
            one = orc.forward(q[b:b + 1, h:h + 1], k[b:b + 1, h:h + 1], v[b:b + 1, h:h + 1], H, W,
                              pool_hw=(p, p), b1=b1[h:h + 1], b2=b2[h:h + 1])
            np.testing.assert_allclose(o[b, h], one[0, 0], atol=0)


def test_linear_in_v_including_dwc():
    H, W, d, p = 4, 4, 3, 2
    r = _rng(21)
    q, k, v1 = _slab(22, H, W, d)
    v2 = r.standard_normal(v1.shape)
    wd = r.standard_normal((1, d, 3, 3))
    f = lambda vv: orc.forward(q[None, None], k[None, None], vv[None, None], H, W,
                               pool_hw=(p, p), dwc_weight=wd)
    np.testing.assert_allclose(f(2.0 * v1 - 0.5 * v2), 2.0 * f(v1) - 0.5 * f(v2), atol=1e-12)


def test_large_logits_are_stable_and_reach_the_argmax_limit():
    H, W, d, p = 4, 4, 6, 2
    q, k, v = _slab(23, H, W, d)
    q, k = q * 50.0, k * 50.0
    o, a, va = orc.forward(q[None, None], k[None, None], v[None, None], H, W, pool_hw=(p, p),
                           return_intermediates=True)
    assert np.all(np.isfinite(o)) and np.all(np.isfinite(va))

    def clear_rows(s):                       # rows whose best logit leads by > 40 (e^-40 ~ 4e-18)
        top2 = np.sort(s, axis=1)[:, -2:]
        return (top2[:, 1] - top2[:, 0]) > 40.0

    s1 = (a[0, 0] @ k.T) / np.sqrt(d)
    ok1 = clear_rows(s1)
    assert ok1.all()                         # the case is built without near-ties in stage 1
    np.testing.assert_allclose(va[0, 0], v[s1.argmax(axis=1)], atol=1e-12)
    s2 = (q @ a[0, 0].T) / np.sqrt(d)
    ok2 = clear_rows(s2)
    assert ok2.sum() >= 12
    np.testing.assert_allclose(o[0, 0][ok2], va[0, 0][s2.argmax(axis=1)][ok2], atol=1e-12)


# ------------------------------------------------------------------------------- Eq. 7
def test_eq7_cost_model_matches_hand_evaluated_fixture():
    vals = {}
    with open(os.path.join(GOLDEN, "eq7_deit_tiny_block.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, val = line.split()
            vals[key] = int(val)
    total, parts = orc.macs(vals["N"], vals["C"], vals["n"], vals["k"])
    assert parts == [vals["proj"], vals["agents"], vals["aggregation"], vals["broadcast"],
                     vals["dwc"]]
    assert total == vals["total"]


def test_threads_do_not_change_the_result():
    B, heads, H, W, d, p = 3, 2, 4, 4, 4, 2
    r = _rng(24)
    q, k, v = (r.standard_normal((B, heads, H * W, d)) for _ in range(3))
    o1 = orc.forward(q, k, v, H, W, pool_hw=(p, p), threads=1)
    o4 = orc.forward(q, k, v, H, W, pool_hw=(p, p), threads=4)
    assert np.array_equal(o1, o4)


# ----------------------------------------------------------------- App. B: bias composition
@pytest.mark.parametrize("h,w,h0,w0", [(14, 14, 7, 7), (8, 12, 3, 5), (9, 7, 9, 7), (16, 16, 1, 1), (5, 6, 2, 9)])
def test_bias_composition_equals_broadcast_plus_library_bilinear_resize(h, w, h0, w0):
    n = 5
    r = _rng(30 + h + w0)
    col, row, blk = r.standard_normal((n, w)), r.standard_normal((n, h)), r.standard_normal((n, h0, w0))
    got = orc.compose_bias(col, row, blk, h, w)
    resized = F.interpolate(torch.from_numpy(blk)[None], size=(h, w), mode="bilinear", align_corners=False)[0].numpy()
    ref = (col[:, None, :] + row[:, :, None] + resized).reshape(n, h * w)
    np.testing.assert_allclose(got, ref, atol=1e-12)
    np.testing.assert_allclose(orc.compose_bias(col, row, blk, h, w, transpose=True), ref.T, atol=1e-12)


def test_bias_composition_closed_forms():
    n, h, w = 3, 6, 4
    r = _rng(31)
    col, row = r.standard_normal((n, w)), r.standard_normal((n, h))
    full = r.standard_normal((n, h, w))
    np.testing.assert_allclose(orc.compose_bias(None, None, full, h, w), full.reshape(n, h * w), atol=1e-14)   # h0 = h: identity
    const = np.tile(np.array([1.5, -2.0, 0.25])[:, None, None], (1, 2, 3))
    np.testing.assert_allclose(orc.compose_bias(None, None, const, h, w), np.repeat(const[:, 0, 0], h * w).reshape(n, -1), atol=1e-14)
    only_col = orc.compose_bias(col, None, None, h, w).reshape(n, h, w)
    for y in range(h):
        np.testing.assert_allclose(only_col[:, y, :], col, atol=0)
    only_row = orc.compose_bias(None, row, None, h, w).reshape(n, h, w)
    for x in range(w):
        np.testing.assert_allclose(only_row[:, :, x], row, atol=0)
    # the module with a composed bias equals the module with the dense bias (the operator takes dense biases)
    q, k, v = _slab(32, h, w, 4)
    blk = r.standard_normal((4, 2, 2))
    b1 = orc.compose_bias(r.standard_normal((4, w)), r.standard_normal((4, h)), blk, h, w)
    o = orc.forward(q[None, None], k[None, None], v[None, None], h, w, pool_hw=(2, 2), b1=b1[None])
    assert np.all(np.isfinite(o))

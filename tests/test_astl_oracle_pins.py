"""Pins for oracle/astl_oracle.py (LayerNorm, GELU, MLP, the layer of Eq. 4 and Eq. 5, and the channel-sliced,
cascaded attention of Eq. 6 / Eq. 8).  The paper prints no worked values for any of these, so they are pinned by
closed forms, identities, loop-written evaluations, an independently pinned routine (the dense attention checker)
and finite differences."""
import math

import numpy as np
import pytest

from oracle import astl_oracle as ao
from oracle import gswa_oracle as orc


# ---------------------------------------------------------------- LayerNorm
def test_layer_norm_closed_forms():
    rng = np.random.default_rng(1)
    C = 12
    g, b = rng.standard_normal(C), rng.standard_normal(C)
    # a constant row has no deviation: only the shift survives
    y, _ = ao.layer_norm(np.full((2, 3, C), 4.25), g, b)
    assert np.abs(y - b).max() < 1e-12
    # a two-valued row: deviations +-h, variance h^2
    lo, hi = -1.5, 2.5
    row = np.array([lo, hi] * (C // 2))
    h = (hi - lo) / 2
    want = np.where(row == hi, 1.0, -1.0) * h / math.sqrt(h * h + ao.LN_EPS) * g + b
    y, _ = ao.layer_norm(row[None], g, b)
    assert np.abs(y[0] - want).max() < 1e-13
    # written out with loops
    x = rng.standard_normal((3, C)) * 3 + 1
    y, _ = ao.layer_norm(x, g, b)
    for t in range(3):
        mu = sum(x[t]) / C
        var = sum((v - mu) ** 2 for v in x[t]) / C
        for c in range(C):
            assert abs(y[t, c] - ((x[t, c] - mu) / math.sqrt(var + ao.LN_EPS) * g[c] + b[c])) < 1e-12
    # without eps the result does not see a positive rescaling or an offset of the row
    y0, _ = ao.layer_norm(x, g, b, eps=0.0)
    y1, _ = ao.layer_norm(7.5 * x - 3.0, g, b, eps=0.0)
    assert np.abs(y0 - y1).max() < 1e-12


def test_layer_norm_backward_finite_differences_and_invariants():
    rng = np.random.default_rng(2)
    C = 10
    x = rng.standard_normal((2, 4, C)) * 2 + 0.5
    g, b = rng.standard_normal(C), rng.standard_normal(C)
    dy = rng.standard_normal(x.shape)
    _, cache = ao.layer_norm(x, g, b)
    dx, dg, db = ao.layer_norm_backward(cache, dy)
    eps = 1e-6
    for name, t, grad in (("x", x, dx), ("g", g, dg), ("b", b, db)):
        for _ in range(3):
            d = rng.standard_normal(t.shape)

            def loss(step):
                args = {"x": x, "g": g, "b": b}
                args[name] = t + step * d
                return float((ao.layer_norm(args["x"], args["g"], args["b"])[0] * dy).sum())
            fd = (loss(eps) - loss(-eps)) / (2 * eps)
            an = float((grad * d).sum())
            assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (name, fd, an)
    # the output ignores the row mean; with eps = 0 it ignores the row scale too
    assert np.abs(dx.sum(-1)).max() < 1e-12
    _, c0 = ao.layer_norm(x, g, b, eps=0.0)
    dx0, _, _ = ao.layer_norm_backward(c0, dy)
    assert np.abs((dx0 * (x - x.mean(-1, keepdims=True))).sum(-1)).max() < 1e-11
    assert np.abs(db - dy.reshape(-1, C).sum(0)).max() < 1e-12


# ---------------------------------------------------------------- GELU, MLP
def test_gelu_values_identities_and_derivative():
    assert ao.gelu(0.0) == 0.0
    # Phi(1) = 0.841344746068543 (standard normal table value)
    assert abs(float(ao.gelu(1.0)) - 0.841344746068543) < 1e-14
    assert abs(float(ao.gelu(-1.0)) + 0.158655253931457) < 1e-14
    x = np.linspace(-6, 6, 49)
    assert np.abs(ao.gelu(x) - ao.gelu(-x) - x).max() < 1e-14          # x Phi(x) + x Phi(-x) = x
    assert abs(float(ao.gelu(12.0)) - 12.0) < 1e-12 and abs(float(ao.gelu(-12.0))) < 1e-12
    assert float(ao.gelu_grad(0.0)) == 0.5
    h = 1e-6
    fd = (ao.gelu(x + h) - ao.gelu(x - h)) / (2 * h)
    assert np.abs(fd - ao.gelu_grad(x)).max() < 1e-9


def test_mlp_against_loops_and_finite_differences():
    rng = np.random.default_rng(3)
    C, Hd = 5, 7
    x = rng.standard_normal((2, 3, C))
    w1, b1 = rng.standard_normal((Hd, C)) * 0.5, rng.standard_normal(Hd) * 0.3
    w2, b2 = rng.standard_normal((C, Hd)) * 0.5, rng.standard_normal(C) * 0.3
    y, cache = ao.mlp_forward(x, w1, b1, w2, b2)
    for idx in np.ndindex(2, 3):
        hid = [sum(w1[j, c] * x[idx][c] for c in range(C)) + b1[j] for j in range(Hd)]
        act = [0.5 * v * (1 + math.erf(v / math.sqrt(2))) for v in hid]
        for c in range(C):
            assert abs(y[idx][c] - (sum(w2[c, j] * act[j] for j in range(Hd)) + b2[c])) < 1e-12
    dy = rng.standard_normal(y.shape)
    grads = dict(zip(("x", "w1", "b1", "w2", "b2"), ao.mlp_backward(cache, dy)))
    tens = {"x": x, "w1": w1, "b1": b1, "w2": w2, "b2": b2}
    eps = 1e-6
    for name, t in tens.items():
        d = rng.standard_normal(t.shape)

        def loss(step):
            a = dict(tens)
            a[name] = t + step * d
            return float((ao.mlp_forward(a["x"], a["w1"], a["b1"], a["w2"], a["b2"])[0] * dy).sum())
        fd = (loss(eps) - loss(-eps)) / (2 * eps)
        an = float((grads[name] * d).sum())
        assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (name, fd, an)


# ---------------------------------------------------------------- channel-sliced heads, cascade
def _sliced_params(rng, C, nh, M, dq):
    ds = C // nh
    return (rng.standard_normal((nh, 2 * dq + ds, ds)) * 0.5, rng.standard_normal((nh, 2 * dq + ds)) * 0.2,
            rng.standard_normal((C, C)) * 0.3, rng.standard_normal(C) * 0.2, rng.standard_normal(((2 * M - 1) ** 2, nh)) * 0.5)


def test_sliced_heads_without_cascade_equal_dense_layer_with_block_diagonal_weights():
    rng = np.random.default_rng(5)
    B, H, W, C, nh, M, dq = 2, 8, 8, 12, 3, 4, 2
    ds = C // nh
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    wh, bh, wp, bp, table = _sliced_params(rng, C, nh, M, dq)
    gh, gs_ = (1, 2), (0, 2)
    y, cache = ao.sliced_forward(x, wh, bh, wp, bp, table, M, gh, gs_, qk_dim=dq, cascade=False)
    g = ao.sliced_backward(cache, dy)
    Cq = nh * dq
    wd = np.zeros((2 * Cq + C, C))
    bd = np.zeros(2 * Cq + C)
    for i in range(nh):
        cols = slice(i * ds, (i + 1) * ds)
        wd[i * dq:(i + 1) * dq, cols] = wh[i, :dq]
        wd[Cq + i * dq:Cq + (i + 1) * dq, cols] = wh[i, dq:2 * dq]
        wd[2 * Cq + i * ds:2 * Cq + (i + 1) * ds, cols] = wh[i, 2 * dq:]
        bd[i * dq:(i + 1) * dq] = bh[i, :dq]
        bd[Cq + i * dq:Cq + (i + 1) * dq] = bh[i, dq:2 * dq]
        bd[2 * Cq + i * ds:2 * Cq + (i + 1) * ds] = bh[i, 2 * dq:]
    yd, cd = orc.forward(x, wd, bd, wp, bp, table, M, gh, gs_, qk_dim=dq, v_dim=ds)
    gd = orc.backward(cd, dy)
    assert np.abs(y - yd).max() < 1e-12
    assert np.abs(g["dx"] - gd["dx"]).max() < 1e-11
    assert np.abs(g["dw_proj"] - gd["dw_proj"]).max() < 1e-11 and np.abs(g["dbias_table"] - gd["dbias_table"]).max() < 1e-11
    for i in range(nh):
        cols = slice(i * ds, (i + 1) * ds)
        assert np.abs(g["dw_heads"][i, :dq] - gd["dw_qkv"][i * dq:(i + 1) * dq, cols]).max() < 1e-11
        assert np.abs(g["dw_heads"][i, 2 * dq:] - gd["dw_qkv"][2 * Cq + i * ds:2 * Cq + (i + 1) * ds, cols]).max() < 1e-11
        assert np.abs(g["db_heads"][i, dq:2 * dq] - gd["db_qkv"][Cq + i * dq:Cq + (i + 1) * dq]).max() < 1e-11


@pytest.mark.parametrize("gh,gs_", [((1, 2), (0, 1)), ((3,), (2,)), ((2, 1), (3, 0))])
def test_cascaded_heads_against_bruteforce_global_attention(gh, gs_):
    rng = np.random.default_rng(7)
    B, H, W, C, nh, M, dq = 1, 8, 8, 6, 3, 4, 3
    x = rng.standard_normal((B, H, W, C))
    prm = _sliced_params(rng, C, nh, M, dq)
    y, _ = ao.sliced_forward(x, *prm, M, gh, gs_, qk_dim=dq, cascade=True)
    yb = ao.sliced_bruteforce(x, *prm, M, gh, gs_, qk_dim=dq, cascade=True)
    assert np.abs(y - yb).max() < 1e-12
    y0, _ = ao.sliced_forward(x, *prm, M, gh, gs_, qk_dim=dq, cascade=False)
    assert np.abs(y - y0).max() > 1e-3                                  # the cascade does something


def test_cascade_passes_nothing_on_from_a_head_whose_value_projection_vanishes():
    rng = np.random.default_rng(9)
    B, H, W, C, nh, M, dq = 1, 8, 8, 8, 4, 4, 2
    ds = C // nh
    x = rng.standard_normal((B, H, W, C))
    wh, bh, wp, bp, table = _sliced_params(rng, C, nh, M, dq)
    wh[1, 2 * dq:] = 0.0
    bh[1, 2 * dq:] = 0.0                                               # head 1 outputs zeros
    eye = np.eye(C)
    a_c, _ = ao.sliced_forward(x, wh, bh, eye, None, table, M, (2, 2), (0, 2), qk_dim=dq, cascade=True)
    a_n, _ = ao.sliced_forward(x, wh, bh, eye, None, table, M, (2, 2), (0, 2), qk_dim=dq, cascade=False)
    assert np.abs(a_c[..., ds:2 * ds]).max() == 0.0
    assert np.abs(a_c[..., 2 * ds:3 * ds] - a_n[..., 2 * ds:3 * ds]).max() < 1e-13      # head 2 saw only its own slice
    assert np.abs(a_c[..., :ds] - a_n[..., :ds]).max() < 1e-13                          # head 0 has no predecessor
    assert np.abs(a_c[..., 3 * ds:] - a_n[..., 3 * ds:]).max() > 1e-3                    # head 3 received head 2's output


def test_cascaded_gradients_match_finite_differences():
    rng = np.random.default_rng(11)
    B, H, W, C, nh, M, dq = 1, 8, 8, 6, 3, 4, 2
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    names = ["w_heads", "b_heads", "w_proj", "b_proj", "bias_table"]
    prm = list(_sliced_params(rng, C, nh, M, dq))
    gh, gs_ = (2, 1), (1, 0)
    _, cache = ao.sliced_forward(x, *prm, M, gh, gs_, qk_dim=dq, cascade=True)
    g = ao.sliced_backward(cache, dy)
    grads = {"x": g["dx"], "w_heads": g["dw_heads"], "b_heads": g["db_heads"], "w_proj": g["dw_proj"], "b_proj": g["db_proj"],
             "bias_table": g["dbias_table"]}
    tens = dict(zip(names, prm))
    tens["x"] = x
    eps = 1e-6
    for name, t in tens.items():
        for _ in range(2):
            d = rng.standard_normal(t.shape)

            def loss(step):
                xx = x + step * d if name == "x" else x
                pp = [p + step * d if n == name else p for n, p in zip(names, prm)]
                return float((ao.sliced_forward(xx, *pp, M, gh, gs_, qk_dim=dq, cascade=True, keep=False)[0] * dy).sum())
            fd = (loss(eps) - loss(-eps)) / (2 * eps)
            an = float((grads[name] * d).sum())
            assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (name, fd, an)


# ---------------------------------------------------------------- the layer
def _astl_params(rng, C, nh, M, Hd):
    return {"ln1_g": 1 + 0.3 * rng.standard_normal(C), "ln1_b": 0.2 * rng.standard_normal(C),
            "w_qkv": rng.standard_normal((3 * C, C)) * 0.3, "b_qkv": rng.standard_normal(3 * C) * 0.2,
            "w_proj": rng.standard_normal((C, C)) * 0.3, "b_proj": rng.standard_normal(C) * 0.2,
            "bias_table": rng.standard_normal(((2 * M - 1) ** 2, nh)) * 0.5,
            "ln2_g": 1 + 0.3 * rng.standard_normal(C), "ln2_b": 0.2 * rng.standard_normal(C),
            "w_fc1": rng.standard_normal((Hd, C)) * 0.4, "b_fc1": rng.standard_normal(Hd) * 0.2,
            "w_fc2": rng.standard_normal((C, Hd)) * 0.4, "b_fc2": rng.standard_normal(C) * 0.2}


def test_layer_structure():
    rng = np.random.default_rng(13)
    B, H, W, C, nh, M, Hd = 1, 8, 8, 8, 2, 4, 12
    x = rng.standard_normal((B, H, W, C))
    p = _astl_params(rng, C, nh, M, Hd)
    x1, _ = ao.astl_forward(x, p, M, (1, 1), (0, 2), with_mlp=False)
    xn, _ = ao.layer_norm(x, p["ln1_g"], p["ln1_b"])
    a, _ = orc.forward(xn, p["w_qkv"], p["b_qkv"], p["w_proj"], p["b_proj"], p["bias_table"], M, (1, 1), (0, 2))
    assert np.abs(x1 - (a + x)).max() < 1e-13                           # Eq. 4
    x2, _ = ao.astl_forward(x, p, M, (1, 1), (0, 2))
    xn2, _ = ao.layer_norm(x1, p["ln2_g"], p["ln2_b"])
    m, _ = ao.mlp_forward(xn2, p["w_fc1"], p["b_fc1"], p["w_fc2"], p["b_fc2"])
    assert np.abs(x2 - (m + x1)).max() < 1e-13                          # Eq. 5
    # a vanishing output projection / second FC layer leaves the skip connection alone
    q = dict(p, w_proj=np.zeros((C, C)), b_proj=np.zeros(C), w_fc2=np.zeros((C, Hd)), b_fc2=np.zeros(C))
    assert np.array_equal(ao.astl_forward(x, q, M, (1, 1), (0, 2))[0], x)


@pytest.mark.parametrize("with_mlp", [False, True])
def test_layer_gradients_match_finite_differences(with_mlp):
    rng = np.random.default_rng(17)
    B, H, W, C, nh, M, Hd = 1, 8, 8, 6, 3, 4, 9
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    p = _astl_params(rng, C, nh, M, Hd)
    gh, gs_ = (2, 1), (0, 2)
    _, cache = ao.astl_forward(x, p, M, gh, gs_, with_mlp=with_mlp)
    g = ao.astl_backward(cache, dy)
    names = [n for n in p if with_mlp or not (n.startswith("ln2") or "fc" in n)]
    eps = 1e-6
    for name in names + ["x"]:
        t = x if name == "x" else p[name]
        for _ in range(2):
            d = rng.standard_normal(t.shape)

            def loss(step):
                xx = x + step * d if name == "x" else x
                pp = dict(p) if name == "x" else dict(p, **{name: t + step * d})
                return float((ao.astl_forward(xx, pp, M, gh, gs_, with_mlp=with_mlp, keep=False)[0] * dy).sum())
            fd = (loss(eps) - loss(-eps)) / (2 * eps)
            an = float((g["dx" if name == "x" else "d" + name] * d).sum())
            assert abs(fd - an) <= 3e-7 * max(1.0, abs(an)), (name, fd, an)

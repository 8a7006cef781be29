"""Pins for the fp64 CPU checker (oracle/gswa_oracle.py).

The paper prints no worked numerical example for the attention layer, so the
checker is pinned by what the mathematics fixes instead: integer identities of
the shift / partition maps, agreement of two independently written forwards,
reduction to textbook softmax attention, exact zeros under the window mask, a
closed form, gradient invariants and finite differences.
"""
import numpy as np
import pytest

from oracle import gswa_oracle as orc


def _params(rng, C, nh, M, bias=True, wstd=0.3):
    w_qkv = rng.standard_normal((3 * C, C)) * wstd
    b_qkv = rng.standard_normal(3 * C) * (0.2 if bias else 0.0)
    w_proj = rng.standard_normal((C, C)) * wstd
    b_proj = rng.standard_normal(C) * (0.2 if bias else 0.0)
    table = rng.standard_normal(((2 * M - 1) ** 2, nh)) * 0.5
    return w_qkv, b_qkv, w_proj, b_proj, table


SHAPES = [(8, 8, 8), (16, 16, 8), (16, 24, 8), (8, 16, 4), (12, 12, 4), (6, 6, 3)]


# ---------------------------------------------------------------- integer maps
@pytest.mark.parametrize("H,W,M", SHAPES)
def test_partition_reverse_and_shift_unshift_are_identities(H, W, M):
    t = np.arange(2 * H * W * 3, dtype=np.float64).reshape(2, H, W, 3)
    assert np.array_equal(orc.window_reverse(orc.window_partition(t, M), M, 2, H, W), t)
    for s in range(M):
        assert np.array_equal(orc.reverse_shift(orc.cyclic_shift(t, s), s), t)
        # direction: shifted[i'] = t[(i'+s) mod H]
        sh = orc.cyclic_shift(t, s)
        assert np.array_equal(sh[:, 0, 0], t[:, s % H, s % W])


@pytest.mark.parametrize("H,W,M", SHAPES)
def test_index_maps_match_roll_and_partition_of_a_token_counter(H, W, M):
    N = M * M
    ids = np.arange(H * W, dtype=np.float64).reshape(1, H, W, 1)
    for s in range(M):
        win, slot, region, rel = orc.index_maps(H, W, M, s)
        # (win, slot) is a bijection onto [0, H*W)
        flat = win.astype(np.int64) * N + slot
        assert np.array_equal(np.sort(flat.ravel()), np.arange(H * W))
        # and it is exactly where roll + partition put each token
        part = orc.window_partition(orc.cyclic_shift(ids, s), M)[..., 0].astype(np.int64)  # [nW,N] -> token id
        assert np.array_equal(part[win.ravel(), slot.ravel()], np.arange(H * W))
        # bias rows
        assert rel.min() == 0 and rel.max() == (2 * M - 1) ** 2 - 1
        assert np.all(np.diag(rel) == (M - 1) * (2 * M - 1) + (M - 1))
        assert rel[0, N - 1] == 0 and rel[N - 1, 0] == (2 * M - 1) ** 2 - 1
        if s == 0:
            assert np.all(region == 0)


@pytest.mark.parametrize("H,W,M", SHAPES)
def test_three_forms_of_the_pair_predicate_agree(H, W, M):
    """same window & same 9-region label == same window & same 2-bit wrap flag == same segment on both axes."""
    ii, jj = np.meshgrid(np.arange(H), np.arange(W), indexing="ij")
    ii, jj = ii.ravel(), jj.ravel()
    for s in range(M):
        win, slot, region, _ = orc.index_maps(H, W, M, s)
        w, r = win.ravel(), region.ravel()
        ip, jp = (ii - s) % H, (jj - s) % W
        wrap = 2 * (ip >= H - s) + (jp >= W - s) if s else np.zeros_like(ip)
        same_w = w[:, None] == w[None, :]
        a = same_w & (r[:, None] == r[None, :])
        b = same_w & (wrap[:, None] == wrap[None, :])
        si, sj = (ii - s) // M, (jj - s) // M
        c = (si[:, None] == si[None, :]) & (sj[:, None] == sj[None, :])
        assert np.array_equal(a, b) and np.array_equal(a, c)
        # inside an allowed pair the slot offset equals the coordinate offset
        sr, sc = slot.ravel() // M, slot.ravel() % M
        p, q = np.nonzero(a)
        assert np.array_equal(sr[p] - sr[q], ii[p] - ii[q]) and np.array_equal(sc[p] - sc[q], jj[p] - jj[q])


# ---------------------------------------------------------------- forward pins
@pytest.mark.parametrize("H,W,M,shifts", [(8, 8, 4, (0, 1)), (8, 8, 4, (2, 3)), (8, 12, 4, (0, 2)), (6, 6, 3, (1, 2)),
                                          (4, 4, 4, (0, 3)), (16, 16, 8, (0, 4))])
def test_procedural_forward_equals_bruteforce_global_attention(H, W, M, shifts):
    rng = np.random.default_rng(11)
    C, nh = 8, 4
    B = 2 if H * W <= 64 else 1
    x = rng.standard_normal((B, H, W, C))
    prm = _params(rng, C, nh, M)
    y, _ = orc.forward(x, *prm, M, (1, 3), shifts)
    yb = orc.bruteforce_forward(x, *prm, M, (1, 3), shifts)
    assert np.abs(y - yb).max() <= 1e-12 * max(1.0, np.abs(yb).max())


def test_every_shift_against_bruteforce_single_group():
    rng = np.random.default_rng(5)
    H, W, M, C, nh = 8, 8, 4, 4, 2
    x = rng.standard_normal((1, H, W, C))
    prm = _params(rng, C, nh, M)
    for s in range(M):
        y, _ = orc.forward(x, *prm, M, (2,), (s,))
        yb = orc.bruteforce_forward(x, *prm, M, (2,), (s,))
        assert np.abs(y - yb).max() <= 1e-12


def test_shift_zero_is_textbook_window_attention():
    """s = 0: each window is softmax(q k^T / sqrt(d) + bias) v, written out directly with loops."""
    rng = np.random.default_rng(3)
    B, H, W, C, nh, M = 2, 8, 12, 6, 3, 4
    d = C // nh
    x = rng.standard_normal((B, H, W, C))
    w_qkv, b_qkv, w_proj, b_proj, table = _params(rng, C, nh, M)
    y, _ = orc.forward(x, w_qkv, b_qkv, w_proj, b_proj, table, M, (nh,), (0,))
    A = np.zeros_like(x)
    for b in range(B):
        for wi in range(H // M):
            for wj in range(W // M):
                coords = [(wi * M + a, wj * M + c) for a in range(M) for c in range(M)]
                X = np.stack([x[b, i, j] for i, j in coords])
                for h in range(nh):
                    q = X @ w_qkv[h * d:(h + 1) * d].T + b_qkv[h * d:(h + 1) * d]
                    k = X @ w_qkv[C + h * d:C + (h + 1) * d].T + b_qkv[C + h * d:C + (h + 1) * d]
                    v = X @ w_qkv[2 * C + h * d:2 * C + (h + 1) * d].T + b_qkv[2 * C + h * d:2 * C + (h + 1) * d]
                    S = q @ k.T / np.sqrt(d)
                    for p, (ia, ja) in enumerate(coords):
                        for r, (ib, jb) in enumerate(coords):
                            S[p, r] += table[(ia - ib + M - 1) * (2 * M - 1) + (ja - jb + M - 1), h]
                    P = np.exp(S - S.max(1, keepdims=True))
                    P /= P.sum(1, keepdims=True)
                    O = P @ v
                    for p, (i, j) in enumerate(coords):
                        A[b, i, j, h * d:(h + 1) * d] = O[p]
    ref = A @ w_proj.T + b_proj
    assert np.abs(y - ref).max() <= 1e-12


def test_masked_weights_are_exactly_zero_and_rows_sum_to_one():
    rng = np.random.default_rng(7)
    B, H, W, C, nh, M, s = 2, 16, 16, 12, 2, 8, 3
    x = rng.standard_normal((B, H, W, C))
    prm = _params(rng, C, nh, M)
    _, cache = orc.forward(x, *prm, M, (1, 1), (0, s))
    P0 = orc.attention_weights(cache, 0)
    P1 = orc.attention_weights(cache, 1)
    assert np.all(P0 > 0)
    assert np.abs(P0.sum(-1) - 1).max() < 1e-14 and np.abs(P1.sum(-1) - 1).max() < 1e-14
    win, slot, region, _ = orc.index_maps(H, W, M, s)
    nW = (H // M) * (W // M)
    lab = np.zeros((nW, M * M), np.int32)
    lab[win.ravel(), slot.ravel()] = region.ravel()
    cross = lab[:, :, None] != lab[:, None, :]                      # [nW,N,N]
    P1 = P1.reshape(B, nW, 1, M * M, M * M)
    assert cross.any()
    for b in range(B):
        assert np.all(P1[b, :, 0][cross] == 0.0)
        assert np.all(P1[b, :, 0][~cross] > 0.0)


def test_closed_form_when_queries_keys_and_table_vanish():
    """W^Q = W^K = 0, b = 0, table = 0  =>  uniform weights: A = mean of v over each segment block."""
    rng = np.random.default_rng(9)
    B, H, W, C, nh, M = 1, 8, 12, 6, 2, 4
    shifts = (0, 1)
    x = rng.standard_normal((B, H, W, C))
    w_qkv, b_qkv, w_proj, b_proj, table = _params(rng, C, nh, M)
    w_qkv[:2 * C] = 0.0
    b_qkv[:2 * C] = 0.0
    table[:] = 0.0
    y, _ = orc.forward(x, w_qkv, b_qkv, w_proj, b_proj, table, M, (1, 1), shifts)
    v = x @ w_qkv[2 * C:].T + b_qkv[2 * C:]
    d = C // nh
    A = np.zeros_like(x)
    for h, s in enumerate(shifts):
        segi = (np.arange(H) - s) // M
        segj = (np.arange(W) - s) // M
        for a in np.unique(segi):
            for c in np.unique(segj):
                blk = np.ix_([0], np.nonzero(segi == a)[0], np.nonzero(segj == c)[0], np.arange(h * d, (h + 1) * d))
                A[blk] = v[blk].mean(axis=(1, 2), keepdims=True)
    ref = A @ w_proj.T + b_proj
    assert np.abs(y - ref).max() <= 1e-13


def test_single_group_special_cases_share_the_code_path():
    """G = 1 with s = 0 / s = M/2 equals the two-group layer restricted to the matching heads."""
    rng = np.random.default_rng(13)
    B, H, W, C, nh, M = 1, 8, 8, 8, 2, 4
    d = C // nh
    x = rng.standard_normal((B, H, W, C))
    w_qkv, b_qkv, w_proj, b_proj, table = _params(rng, C, nh, M)
    eye = np.eye(C)
    zero = np.zeros(C)
    a_mixed, _ = orc.forward(x, w_qkv, b_qkv, eye, zero, table, M, (1, 1), (0, 2))
    a_plain, _ = orc.forward(x, w_qkv, b_qkv, eye, zero, table, M, (2,), (0,))
    a_shift, _ = orc.forward(x, w_qkv, b_qkv, eye, zero, table, M, (2,), (2,))
    assert np.abs(a_mixed[..., :d] - a_plain[..., :d]).max() < 1e-14
    assert np.abs(a_mixed[..., d:] - a_shift[..., d:]).max() < 1e-14
    assert not np.allclose(a_plain[..., d:], a_shift[..., d:])


def test_batch_items_are_independent():
    rng = np.random.default_rng(17)
    B, H, W, C, nh, M = 3, 8, 8, 8, 2, 4
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    prm = _params(rng, C, nh, M)
    y, cache = orc.forward(x, *prm, M, (1, 1), (0, 2))
    g = orc.backward(cache, dy)
    perm = np.array([2, 0, 1])
    y2, cache2 = orc.forward(x[perm], *prm, M, (1, 1), (0, 2))
    g2 = orc.backward(cache2, dy[perm])
    assert np.allclose(y2, y[perm], atol=1e-13) and np.allclose(g2["dx"], g["dx"][perm], atol=1e-13)
    for n in ("dw_qkv", "db_qkv", "dw_proj", "db_proj", "dbias_table"):
        assert np.allclose(g2[n], g[n], atol=1e-11)
    yc, gc = orc.forward_backward_chunked(x, *prm, M, (1, 1), (0, 2), dy, chunk=2)
    assert np.allclose(yc, y, atol=1e-13)
    for n in g:
        assert np.allclose(gc[n], g[n], atol=1e-11)


# ---------------------------------------------------------------- gradient pins
def _loss(x, prm, M, gh, gs, dy):
    y, _ = orc.forward(x, *prm, M, gh, gs, keep=False)
    return float((y * dy).sum())


@pytest.mark.parametrize("H,W,M,gh,gs", [(8, 8, 4, (1, 1), (0, 2)), (8, 12, 4, (2, 1), (3, 1)), (6, 6, 3, (3,), (2,)),
                                         (16, 16, 8, (1, 1), (0, 4))])
def test_gradients_match_central_finite_differences(H, W, M, gh, gs):
    rng = np.random.default_rng(23)
    nh = sum(gh)
    C = 2 * nh
    B = 2 if H * W < 200 else 1
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    prm = list(_params(rng, C, nh, M))
    y, cache = orc.forward(x, *prm, M, gh, gs)
    g = orc.backward(cache, dy)
    names = ["w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table"]
    grads = {"x": g["dx"], "w_qkv": g["dw_qkv"], "b_qkv": g["db_qkv"], "w_proj": g["dw_proj"], "b_proj": g["db_proj"],
             "bias_table": g["dbias_table"]}
    eps = 1e-6

    def directional(name, direction):
        def at(t):
            xx = x + t * direction if name == "x" else x
            pp = [p + t * direction if n == name else p for n, p in zip(names, prm)]
            return _loss(xx, pp, M, gh, gs, dy)
        return (at(eps) - at(-eps)) / (2 * eps)

    tensors = dict(zip(names, prm))
    tensors["x"] = x
    for name, t in tensors.items():
        for _ in range(2):                                           # random directions
            dirn = rng.standard_normal(t.shape)
            fd = directional(name, dirn)
            an = float((grads[name] * dirn).sum())
            assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (name, fd, an)
    # single coordinates: border strips of x, rarely used table corners, a q-row and a k-row of w_qkv
    T2 = (2 * M - 1) ** 2
    singles = [("x", (0, 0, 0, 0)), ("x", (B - 1, H - 1, W - 1, C - 1)), ("x", (0, H - 1, 0, 1)),
               ("bias_table", (0, 0)), ("bias_table", (T2 - 1, nh - 1)), ("bias_table", (2 * M - 2, 0)),
               ("bias_table", ((M - 1) * (2 * M - 1) + M - 1, nh - 1)),
               ("w_qkv", (0, 1)), ("w_qkv", (C + 1, 0)), ("w_qkv", (3 * C - 1, C - 1)), ("b_qkv", (2 * C,))]
    for name, idx in singles:
        dirn = np.zeros(tensors[name].shape)
        dirn[idx] = 1.0
        fd = directional(name, dirn)
        an = float(grads[name][idx])
        assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (name, idx, fd, an)


def test_gradient_invariants():
    rng = np.random.default_rng(29)
    B, H, W, C, nh, M = 2, 8, 8, 12, 3, 4
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    prm = _params(rng, C, nh, M)
    _, cache = orc.forward(x, *prm, M, (1, 2), (0, 2))
    g = orc.backward(cache, dy)
    # softmax is invariant to a constant added to a whole score row -> each head's table gradient sums to 0
    assert np.abs(g["dbias_table"].sum(axis=0)).max() < 1e-12
    # ... and to a constant vector added to every key -> the k slice of b_qkv has zero gradient
    assert np.abs(g["db_qkv"][C:2 * C]).max() < 1e-12
    assert np.allclose(g["db_proj"], dy.reshape(-1, C).sum(0), atol=1e-12)
    assert np.abs(g["db_qkv"][:C]).max() > 1e-3 and np.abs(g["db_qkv"][2 * C:]).max() > 1e-3


# ---------------------------------------------------------------- narrowed Q/K projections (Sec. "Parameter Allocation")
def _narrow_params(rng, C, nh, M, dq, dv, wstd=0.3):
    Cq, Cv = nh * dq, nh * dv
    return (rng.standard_normal((2 * Cq + Cv, C)) * wstd, rng.standard_normal(2 * Cq + Cv) * 0.2,
            rng.standard_normal((C, Cv)) * wstd, rng.standard_normal(C) * 0.2, rng.standard_normal(((2 * M - 1) ** 2, nh)) * 0.5)


@pytest.mark.parametrize("dq,dv", [(1, 2), (3, 2), (2, 5)])
def test_narrow_projections_against_bruteforce_global_attention(dq, dv):
    rng = np.random.default_rng(31)
    B, H, W, C, nh, M = 1, 8, 8, 8, 4, 4
    x = rng.standard_normal((B, H, W, C))
    prm = _narrow_params(rng, C, nh, M, dq, dv)
    y, _ = orc.forward(x, *prm, M, (1, 3), (0, 1), qk_dim=dq, v_dim=dv)
    yb = orc.bruteforce_forward(x, *prm, M, (1, 3), (0, 1), qk_dim=dq, v_dim=dv)
    assert y.shape == x.shape
    assert np.abs(y - yb).max() <= 1e-12 * max(1.0, np.abs(yb).max())


def test_narrow_layer_equals_full_width_layer_with_zero_rows():
    """A layer with qk_dim = k < d is the full-width layer whose Q,K rows beyond k are zero and whose Q rows are
    rescaled by sqrt(d / k) (the full layer divides the scores by sqrt(d), the narrow one by sqrt(k)).  The
    gradients of the shared rows agree likewise (those of the rescaled Q rows up to that factor)."""
    rng = np.random.default_rng(37)
    B, H, W, C, nh, M, k = 2, 8, 8, 12, 3, 4, 2
    d = C // nh
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    w, b, wp, bp, table = _narrow_params(rng, C, nh, M, k, d)
    Cq = nh * k
    full_w = np.zeros((3 * C, C))
    full_b = np.zeros(3 * C)
    f = np.sqrt(d / k)
    rows_q, rows_k = [], []
    for h in range(nh):
        for c in range(k):
            rows_q.append(h * d + c)
            rows_k.append(C + h * d + c)
    full_w[rows_q] = w[:Cq] * f
    full_b[rows_q] = b[:Cq] * f
    full_w[rows_k] = w[Cq:2 * Cq]
    full_b[rows_k] = b[Cq:2 * Cq]
    full_w[2 * C:] = w[2 * Cq:]
    full_b[2 * C:] = b[2 * Cq:]
    gh, gs = (1, 2), (0, 2)
    y, cache = orc.forward(x, w, b, wp, bp, table, M, gh, gs, qk_dim=k)
    g = orc.backward(cache, dy)
    yf, cachef = orc.forward(x, full_w, full_b, wp, bp, table, M, gh, gs)
    gf = orc.backward(cachef, dy)
    assert np.abs(y - yf).max() <= 1e-13
    assert np.abs(g["dx"] - gf["dx"]).max() <= 1e-12
    assert np.abs(g["dw_qkv"][:Cq] - gf["dw_qkv"][rows_q] * f).max() <= 1e-11
    assert np.abs(g["dw_qkv"][Cq:2 * Cq] - gf["dw_qkv"][rows_k]).max() <= 1e-11
    assert np.abs(g["dw_qkv"][2 * Cq:] - gf["dw_qkv"][2 * C:]).max() <= 1e-11
    assert np.abs(g["db_qkv"][:Cq] - gf["db_qkv"][rows_q] * f).max() <= 1e-11
    assert np.abs(g["dbias_table"] - gf["dbias_table"]).max() <= 1e-11
    assert np.abs(g["dw_proj"] - gf["dw_proj"]).max() <= 1e-11


def test_narrow_projection_gradients_match_finite_differences():
    rng = np.random.default_rng(41)
    B, H, W, C, nh, M, dq, dv = 1, 8, 8, 6, 3, 4, 3, 4
    x = rng.standard_normal((B, H, W, C))
    dy = rng.standard_normal((B, H, W, C))
    prm = list(_narrow_params(rng, C, nh, M, dq, dv))
    gh, gs = (2, 1), (1, 0)
    _, cache = orc.forward(x, *prm, M, gh, gs, qk_dim=dq, v_dim=dv)
    g = orc.backward(cache, dy)
    names = ["w_qkv", "b_qkv", "w_proj", "b_proj", "bias_table"]
    grads = {"x": g["dx"], "w_qkv": g["dw_qkv"], "b_qkv": g["db_qkv"], "w_proj": g["dw_proj"], "b_proj": g["db_proj"],
             "bias_table": g["dbias_table"]}
    tensors = dict(zip(names, prm))
    tensors["x"] = x
    eps = 1e-6
    for name, t in tensors.items():
        for _ in range(2):
            dirn = rng.standard_normal(t.shape)

            def at(step):
                xx = x + step * dirn if name == "x" else x
                pp = [p + step * dirn if n == name else p for n, p in zip(names, prm)]
                yy, _ = orc.forward(xx, *pp, M, gh, gs, keep=False, qk_dim=dq, v_dim=dv)
                return float((yy * dy).sum())
            fd = (at(eps) - at(-eps)) / (2 * eps)
            an = float((grads[name] * dirn).sum())
            assert abs(fd - an) <= 2e-7 * max(1.0, abs(an)), (name, fd, an)

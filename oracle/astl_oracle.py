"""fp64 CPU checker for the Agile Swin Transformer Layer (ASTL) around GSWA, and for the channel-sliced,
cascaded form of GSWA.

TEST INFRASTRUCTURE ONLY (see gswa_oracle.py: same rules).  numpy float64 throughout; builds on the
attention checker of gswa_oracle.py for the attention itself and adds what the layer puts around it.

What it computes (AgileIR, Sec. "Agile Swin Transformer Block", Eq. 4 and Eq. 5):
    X1 = GSWA(LN(X)) + X
    X2 = MLP(LN(X1)) + X1
with LayerNorm over the channels of each token, and an MLP of two fully-connected layers with a GELU
between them.  Readings where the paper is silent: LayerNorm adds eps = 1e-5 to the variance (biased
variance over the C channels) and has a learnable scale and shift; GELU is the exact Gaussian-CDF form
x * Phi(x); the hidden width is a free parameter (rows of w_fc1).

Sec. "Group Shifted Window Attention", Eq. 6 read literally, and Eq. 8 (`sliced_forward`): the input is
split into h channel slices X_i of C/h channels, head i projects only its own slice
(W_i^Q, W_i^K: [dq, C/h]; W_i^V: [C/h, C/h]) and attends inside its group's (shifted) windows; with the
cascade, the input of head i >= 2 is X_i plus the OUTPUT of head i-1 ("each X_i result is accumulated
from the former head", which is only well-typed as an addition to the next head's input, the printed
equation being circular); the heads' outputs are concatenated and projected by W^P (Eq. 7).

Parity pins (tests/test_astl_oracle_pins.py): LayerNorm closed forms (constant row -> shift only;
two-valued rows -> +-scale; invariance to an affine change of the row), GELU values and symmetry
identities, the MLP against a loop-written evaluation, finite differences of every gradient, the sliced
layer without cascade against the dense checker with block-diagonal weights, the cascaded layer against a
brute-force evaluation head by head, and cascade invariants (a head whose W^V vanishes passes nothing on).
"""
from __future__ import annotations

import math

import numpy as np

from . import gswa_oracle as gs

F64 = np.float64
LN_EPS = 1e-5


# --------------------------------------------------------------------------
# LayerNorm over the last axis (Eq. 4, Eq. 5: "LayerNorm layer is placed before GSWA and MLP")
# --------------------------------------------------------------------------
def layer_norm(x, gamma, beta, eps=LN_EPS):
    x = np.asarray(x, F64)
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    rstd = 1.0 / np.sqrt(var + eps)
    xhat = (x - mu) * rstd
    return xhat * np.asarray(gamma, F64) + np.asarray(beta, F64), (xhat, rstd, np.asarray(gamma, F64))


def layer_norm_backward(cache, dy):
    xhat, rstd, gamma = cache
    dy = np.asarray(dy, F64)
    C = xhat.shape[-1]
    dxhat = dy * gamma
    dx = rstd * (dxhat - dxhat.mean(axis=-1, keepdims=True) - xhat * (dxhat * xhat).mean(axis=-1, keepdims=True))
    return dx, (dy * xhat).reshape(-1, C).sum(axis=0), dy.reshape(-1, C).sum(axis=0)


# --------------------------------------------------------------------------
# GELU (exact form) and the MLP
# --------------------------------------------------------------------------
_erf = np.vectorize(math.erf, otypes=[F64])


def gelu(x):
    x = np.asarray(x, F64)
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def gelu_grad(x):
    x = np.asarray(x, F64)
    return 0.5 * (1.0 + _erf(x / math.sqrt(2.0))) + x * np.exp(-0.5 * x * x) / math.sqrt(2.0 * math.pi)


def mlp_forward(x, w1, b1, w2, b2):
    """fc2(GELU(fc1(x))); w1 [hidden, C], w2 [C, hidden]."""
    x = np.asarray(x, F64)
    h = x @ np.asarray(w1, F64).T + np.asarray(b1, F64)
    a = gelu(h)
    return a @ np.asarray(w2, F64).T + np.asarray(b2, F64), (x, h, a, np.asarray(w1, F64), np.asarray(w2, F64))


def mlp_backward(cache, dy):
    x, h, a, w1, w2 = cache
    dy = np.asarray(dy, F64)
    C, Hd = x.shape[-1], h.shape[-1]
    dy2 = dy.reshape(-1, C)
    dw2 = dy2.T @ a.reshape(-1, Hd)
    db2 = dy2.sum(axis=0)
    dh = (dy @ w2) * gelu_grad(h)
    dh2 = dh.reshape(-1, Hd)
    dw1 = dh2.T @ x.reshape(-1, C)
    db1 = dh2.sum(axis=0)
    return dh @ w1, dw1, db1, dw2, db2


# --------------------------------------------------------------------------
# channel-sliced heads with the cascade (Eq. 6 literal, Eq. 8)
# --------------------------------------------------------------------------
def _head_shifts(group_heads, group_shift):
    return [s for gh, s in zip(group_heads, group_shift) for _ in range(gh)]


def sliced_forward(x, w_heads, b_heads, w_proj, b_proj, table, M, group_heads, group_shift, qk_dim=None, cascade=True,
                   keep=True):
    """Channel-sliced GSWA.  w_heads [h, 2*dq + ds, ds] and b_heads [h, 2*dq + ds] hold, per head, the rows
    q | k | v of its projections of the head's ds = C/h input channels (v keeps the slice width, so that a head's
    output can be added to the next head's input).  Returns y [B,H,W,C] and a cache."""
    x = np.asarray(x, F64)
    w_heads = np.asarray(w_heads, F64)
    b_heads = np.asarray(b_heads, F64)
    w_proj = np.asarray(w_proj, F64)
    table = np.asarray(table, F64)
    B, H, W, C = x.shape
    nh = int(sum(group_heads))
    ds = C // nh
    dq = int(qk_dim) if qk_dim else ds
    assert C % nh == 0 and w_heads.shape == (nh, 2 * dq + ds, ds) and w_proj.shape == (C, C)
    b_proj = np.zeros(C, F64) if b_proj is None else np.asarray(b_proj, F64)
    shifts = _head_shifts(group_heads, group_shift)
    eye, zero = np.eye(ds), np.zeros(ds)
    outs, caches = [], []
    prev = None
    for i in range(nh):
        xi = x[..., i * ds:(i + 1) * ds]
        if cascade and prev is not None:
            xi = xi + prev                                   # Eq. 8: the former head's output joins this head's input
        # one head = a one-head GSWA layer on the slice with an identity output projection
        o, c = gs.forward(xi, w_heads[i], b_heads[i], eye, zero, table[:, i:i + 1], M, (1,), (shifts[i],), keep=keep,
                          qk_dim=dq, v_dim=ds)
        outs.append(o)
        caches.append(c)
        prev = o
    A = np.concatenate(outs, axis=-1)                        # Eq. 7: concatenate, then W^P
    y = A @ w_proj.T + b_proj
    cache = dict(caches=caches, A=A, w_proj=w_proj, cascade=cascade, ds=ds, nh=nh, table_shape=table.shape) if keep else None
    return y, cache


def sliced_backward(cache, dy):
    """-> dict(dx, dw_heads, db_heads, dw_proj, db_proj, dbias_table)."""
    dy = np.asarray(dy, F64)
    A, w_proj, ds, nh = cache["A"], cache["w_proj"], cache["ds"], cache["nh"]
    C = A.shape[-1]
    dy2 = dy.reshape(-1, C)
    dw_proj = dy2.T @ A.reshape(-1, C)
    db_proj = dy2.sum(axis=0)
    dA = dy @ w_proj
    dx = np.zeros_like(A)
    dws, dbs = [None] * nh, [None] * nh
    dtable = np.zeros(cache["table_shape"], F64)
    carry = None                                             # gradient flowing back into head i's output from head i+1's input
    for i in reversed(range(nh)):
        do = dA[..., i * ds:(i + 1) * ds]
        if carry is not None:
            do = do + carry
        g = gs.backward(cache["caches"][i], do)
        dx[..., i * ds:(i + 1) * ds] = g["dx"]
        dws[i], dbs[i] = g["dw_qkv"], g["db_qkv"]
        dtable[:, i] = g["dbias_table"][:, 0]
        carry = g["dx"] if cache["cascade"] else None        # head i's input contained head i-1's output
    return dict(dx=dx, dw_heads=np.stack(dws), db_heads=np.stack(dbs), dw_proj=dw_proj, db_proj=db_proj, dbias_table=dtable)


def sliced_bruteforce(x, w_heads, b_heads, w_proj, b_proj, table, M, group_heads, group_shift, qk_dim=None, cascade=True):
    """The same layer by masked global attention head by head (loops; tiny inputs only)."""
    x = np.asarray(x, F64)
    w_heads = np.asarray(w_heads, F64)
    B, H, W, C = x.shape
    nh = int(sum(group_heads))
    ds = C // nh
    dq = int(qk_dim) if qk_dim else ds
    shifts = _head_shifts(group_heads, group_shift)
    outs, prev = [], None
    for i in range(nh):
        xi = x[..., i * ds:(i + 1) * ds] + (prev if (cascade and prev is not None) else 0.0)
        o = gs.bruteforce_forward(xi, w_heads[i], np.asarray(b_heads, F64)[i], np.eye(ds), np.zeros(ds), np.asarray(table, F64)[:, i:i + 1],
                                  M, (1,), (shifts[i],), qk_dim=dq, v_dim=ds)
        outs.append(o)
        prev = o
    b_proj = np.zeros(C) if b_proj is None else np.asarray(b_proj, F64)
    return np.concatenate(outs, axis=-1) @ np.asarray(w_proj, F64).T + b_proj


# --------------------------------------------------------------------------
# the layer (Eq. 4, Eq. 5)
# --------------------------------------------------------------------------
def astl_forward(x, p, M, group_heads, group_shift, qk_dim=None, v_dim=None, with_mlp=True, keep=True):
    """p: dict with ln1_g, ln1_b, w_qkv, b_qkv, w_proj, b_proj, bias_table and, with the MLP, ln2_g, ln2_b,
    w_fc1, b_fc1, w_fc2, b_fc2.  Returns the layer output and a cache."""
    x = np.asarray(x, F64)
    xn, c_ln1 = layer_norm(x, p["ln1_g"], p["ln1_b"])
    a, c_attn = gs.forward(xn, p["w_qkv"], p["b_qkv"], p["w_proj"], p["b_proj"], p["bias_table"], M, group_heads, group_shift,
                           keep=keep, qk_dim=qk_dim, v_dim=v_dim)
    x1 = a + x                                               # Eq. 4
    if not with_mlp:
        return x1, (dict(ln1=c_ln1, attn=c_attn, mlp=None) if keep else None)
    xn2, c_ln2 = layer_norm(x1, p["ln2_g"], p["ln2_b"])
    m, c_mlp = mlp_forward(xn2, p["w_fc1"], p["b_fc1"], p["w_fc2"], p["b_fc2"])
    x2 = m + x1                                              # Eq. 5
    return x2, (dict(ln1=c_ln1, attn=c_attn, ln2=c_ln2, mlp=c_mlp) if keep else None)


def astl_backward(cache, dy):
    """Gradients of <out, dy>: dict with dx and d<name> for every parameter of astl_forward."""
    dy = np.asarray(dy, F64)
    g = {}
    dx1 = dy
    if cache["mlp"] is not None:
        dxn2, g["dw_fc1"], g["db_fc1"], g["dw_fc2"], g["db_fc2"] = mlp_backward(cache["mlp"], dy)
        dres, g["dln2_g"], g["dln2_b"] = layer_norm_backward(cache["ln2"], dxn2)
        dx1 = dy + dres                                      # skip connection of Eq. 5
    ga = gs.backward(cache["attn"], dx1)
    for n in ("dw_qkv", "db_qkv", "dw_proj", "db_proj", "dbias_table"):
        g[n] = ga[n]
    dres, g["dln1_g"], g["dln1_b"] = layer_norm_backward(cache["ln1"], ga["dx"])
    g["dx"] = dx1 + dres                                     # skip connection of Eq. 4
    return g

"""fp64 CPU checker for Group Shifted Window Attention (GSWA), forward and backward.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is compared against.  It shares no code with the CUDA path and is
imported only by the tests, the smoke check and the benchmark's CPU-baseline
leg.  numpy float64 throughout.

What it computes (AgileIR, Sec. "Group Shifted Window Attention"):
  * Eq. 6: per head, Attn(X W^Q, X W^K, X W^V) inside M x M windows
    (Sec. "Patch Embedding": H x W x C -> HW/M^2 x M^2 x C).  The paper does
    not spell Attn out; the reading taken is the shifted-window attention it
    decomposes: softmax(Q K^T / sqrt(d) + B + mask) V, softmax over keys.
  * heads are split into consecutive groups; a group with shift s > 0 sees the
    feature map cyclically shifted by s with the window mask applied
    (GSW-MSA), a group with s = 0 sees plain windows (GW-MSA).
  * Sec. "Learnable Relative Shifted Bias": B in R^{(2M-1)x(2M-1)}, one column
    of a [(2M-1)^2, heads] table per head, indexed by slot offsets in the
    window frame (so it moves with the shifted windows).
  * Eq. 7: concatenate heads, multiply by W^P.
Two independently written forwards are kept: `forward` walks the paper's steps
(shift, partition, mask, attention, reverse), `bruteforce_forward` evaluates
masked attention over all H*W tokens of an image in original coordinates and
never rolls or partitions anything.  `backward` is hand-derived reverse mode of
`forward`.

Parity pins (tests/test_oracle_*.py): the two forwards agree; shift 0 reduces
to textbook per-window softmax attention; partition/reverse and shift/unshift
are identities; masked weights are exactly 0; a closed form when Q,K and the
table vanish; gradient invariants; central finite differences.  The paper
prints no worked numerical example, so no printed values are pinned.

Sec. "Parameter Allocation" (Q and K projections narrower than V): optional per-head
widths `qk_dim`, `v_dim`; the scores are then scaled by qk_dim^-1/2.  Pinned by the same
pins run at qk_dim != v_dim and by the identity "a narrow layer equals the full-width
layer whose extra Q,K rows are zero and whose Q rows are rescaled by sqrt(d / qk_dim)".

Conventions fixed where the paper is silent:
  x[B,H,W,C] channels last; w_qkv[3C,C] rows ordered [q|k|v], head-major
  inside each; y = x W^T + b; cyclic shift reads from +s
  (shifted[i'] = x[(i'+s) mod H]); mask value is -inf.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# integer maps (Sec. "Patch Embedding"; shift and window mask of GSW-MSA)
# --------------------------------------------------------------------------
def axis_region(n: int, M: int, s: int) -> np.ndarray:
    """Region label along one axis of the shifted frame: [0,n-M) -> 0, [n-M,n-s) -> 1, [n-s,n) -> 2."""
    r = np.zeros(n, dtype=np.int32)
    if s > 0:
        r[n - M:n - s] = 1
        r[n - s:] = 2
    return r


def index_maps(H: int, W: int, M: int, s: int):
    """Maps of one image for shift s.

    Returns (win, slot, region, rel):
      win[i,j]    window number (row-major over the H/M x W/M grid of the shifted frame) of ORIGINAL token (i,j)
      slot[i,j]   position inside that window, row-major over M x M
      region[i,j] 3*r(i') + r(j') label of the window mask (all 0 when s == 0)
      rel[p,q]    row of the bias table used for query slot p and key slot q
    """
    i = np.arange(H)[:, None]
    j = np.arange(W)[None, :]
    ip = (i - s) % H            # where original row i lands in the shifted frame
    jp = (j - s) % W
    win = (ip // M) * (W // M) + (jp // M)
    slot = (ip % M) * M + (jp % M)
    ri = axis_region(H, M, s)
    rj = axis_region(W, M, s)
    region = 3 * ri[ip] + rj[jp]
    a = np.arange(M * M) // M
    c = np.arange(M * M) % M
    rel = (a[:, None] - a[None, :] + M - 1) * (2 * M - 1) + (c[:, None] - c[None, :] + M - 1)
    return win.astype(np.int32), slot.astype(np.int32), region.astype(np.int32), rel.astype(np.int32)


def cyclic_shift(t: np.ndarray, s: int) -> np.ndarray:
    """shifted[b,i',j'] = t[b,(i'+s) mod H,(j'+s) mod W]."""
    return np.roll(t, shift=(-s, -s), axis=(1, 2)) if s else t


def reverse_shift(t: np.ndarray, s: int) -> np.ndarray:
    return np.roll(t, shift=(s, s), axis=(1, 2)) if s else t


def window_partition(t: np.ndarray, M: int) -> np.ndarray:
    """[B,H,W,c] -> [B*HW/M^2, M^2, c]."""
    B, H, W, c = t.shape
    t = t.reshape(B, H // M, M, W // M, M, c).transpose(0, 1, 3, 2, 4, 5)
    return t.reshape(B * (H // M) * (W // M), M * M, c)


def window_reverse(w: np.ndarray, M: int, B: int, H: int, W: int) -> np.ndarray:
    c = w.shape[-1]
    t = w.reshape(B, H // M, W // M, M, M, c).transpose(0, 1, 3, 2, 4, 5)
    return t.reshape(B, H, W, c)


def window_mask(H: int, W: int, M: int, s: int) -> np.ndarray:
    """Additive mask [HW/M^2, M^2, M^2]: 0 where query and key carry the same region label, -inf elsewhere."""
    ri = axis_region(H, M, s)
    rj = axis_region(W, M, s)
    lab = (3 * ri[:, None] + rj[None, :]).astype(F64)[None, :, :, None]
    lw = window_partition(lab, M)[..., 0]                      # [nW, N]
    same = lw[:, :, None] == lw[:, None, :]
    return np.where(same, 0.0, -np.inf)


# --------------------------------------------------------------------------
# forward, procedural (Eq. 6, Eq. 7)
# --------------------------------------------------------------------------
def _check(x, group_heads, group_shift, M):
    B, H, W, C = x.shape
    nh = int(sum(group_heads))
    assert len(group_heads) == len(group_shift) and nh > 0 and C % nh == 0
    assert H % M == 0 and W % M == 0
    assert all(0 <= s < M for s in group_shift)
    return B, H, W, C, nh, C // nh


def _widths(d, qk_dim, v_dim):
    """Per-head widths of Q,K and of V (Sec. "Parameter Allocation": Q and K may be narrower than V; both
    default to the head dim C / heads)."""
    return (int(qk_dim) if qk_dim else d), (int(v_dim) if v_dim else d)


def forward(x, w_qkv, b_qkv, w_proj, b_proj, table, M, group_heads, group_shift, keep=True, qk_dim=None, v_dim=None):
    """y[B,H,W,C] and a cache for `backward`.  All arguments are converted to float64.

    With per-head widths dq = qk_dim and dv = v_dim (Sec. "Parameter Allocation"): w_qkv is
    [2*heads*dq + heads*dv, C] with rows q | k | v (head-major inside each), w_proj is [C, heads*dv], and the
    scores are scaled by dq^-1/2."""
    x = np.asarray(x, F64)
    w_qkv = np.asarray(w_qkv, F64)
    w_proj = np.asarray(w_proj, F64)
    table = np.asarray(table, F64)
    B, H, W, C, nh, d = _check(x, group_heads, group_shift, M)
    dq, dv = _widths(d, qk_dim, v_dim)
    Cq, Cv = nh * dq, nh * dv
    assert w_qkv.shape == (2 * Cq + Cv, C) and w_proj.shape == (C, Cv)
    b_qkv = np.zeros(2 * Cq + Cv, F64) if b_qkv is None else np.asarray(b_qkv, F64)
    b_proj = np.zeros(C, F64) if b_proj is None else np.asarray(b_proj, F64)
    N = M * M
    scale = float(dq) ** -0.5

    qkv = x @ w_qkv.T + b_qkv                                   # Eq. 6 projections
    q = qkv[..., 0:Cq] * scale
    k = qkv[..., Cq:2 * Cq]
    v = qkv[..., 2 * Cq:2 * Cq + Cv]
    rel = index_maps(H, W, M, 0)[3]

    A = np.zeros((B, H, W, Cv), F64)
    groups = []
    h0 = 0
    for gh, s in zip(group_heads, group_shift):
        chq = slice(h0 * dq, (h0 + gh) * dq)
        ch = slice(h0 * dv, (h0 + gh) * dv)
        qw = window_partition(cyclic_shift(q[..., chq], s), M).reshape(-1, N, gh, dq)
        kw = window_partition(cyclic_shift(k[..., chq], s), M).reshape(-1, N, gh, dq)
        vw = window_partition(cyclic_shift(v[..., ch], s), M).reshape(-1, N, gh, dv)
        S = np.einsum("nphd,nqhd->nhpq", qw, kw)
        S = S + table[rel][:, :, h0:h0 + gh].transpose(2, 0, 1)[None]      # bias B
        if s > 0:
            nW = (H // M) * (W // M)
            mask = window_mask(H, W, M, s)                                  # [nW,N,N]
            S = (S.reshape(B, nW, gh, N, N) + mask[None, :, None]).reshape(B * nW, gh, N, N)
        Smax = S.max(axis=-1, keepdims=True)
        E = np.exp(S - Smax)
        P = E / E.sum(axis=-1, keepdims=True)
        O = np.einsum("nhpq,nqhd->nphd", P, vw).reshape(-1, N, gh * dv)
        A[..., ch] = reverse_shift(window_reverse(O, M, B, H, W), s)        # concat of Eq. 7
        groups.append((ch, s, qw, kw, vw, P, chq) if keep else None)
        h0 += gh
    y = A @ w_proj.T + b_proj                                               # W^P of Eq. 7
    cache = dict(x=x, w_qkv=w_qkv, w_proj=w_proj, table_shape=table.shape, M=M, group_heads=tuple(group_heads),
                 group_shift=tuple(group_shift), A=A, groups=groups, rel=rel, scale=scale) if keep else None
    return y, cache


def attention_weights(cache, group: int) -> np.ndarray:
    """P[B*nW, heads_in_group, N, N] of one group, for tests."""
    return cache["groups"][group][5]


# --------------------------------------------------------------------------
# backward (reverse mode of the forward above)
# --------------------------------------------------------------------------
def backward(cache, dy):
    """Gradients of <y, dy> w.r.t. x and every parameter.

    Returns dict(dx, dw_qkv, db_qkv, dw_proj, db_proj, dbias_table).
    """
    dy = np.asarray(dy, F64)
    x, w_qkv, w_proj = cache["x"], cache["w_qkv"], cache["w_proj"]
    M, rel, scale, A = cache["M"], cache["rel"], cache["scale"], cache["A"]
    B, H, W, C = x.shape
    N = M * M
    dy2 = dy.reshape(-1, C)
    dw_proj = dy2.T @ A.reshape(-1, A.shape[-1])
    db_proj = dy2.sum(axis=0)
    dA = dy @ w_proj

    nh = int(sum(cache["group_heads"]))
    wq, wv = cache["groups"][0][2].shape[-1], cache["groups"][0][4].shape[-1]   # per-head widths of q,k and of v
    dq = np.zeros((B, H, W, nh * wq), F64)
    dk = np.zeros((B, H, W, nh * wq), F64)
    dv = np.zeros((B, H, W, nh * wv), F64)
    dtable = np.zeros(cache["table_shape"], F64)
    h0 = 0
    for (ch, s, qw, kw, vw, P, chq), gh in zip(cache["groups"], cache["group_heads"]):
        dO = window_partition(cyclic_shift(dA[..., ch], s), M).reshape(-1, N, gh, wv)
        dvw = np.einsum("nhpq,nphd->nqhd", P, dO)
        dP = np.einsum("nphd,nqhd->nhpq", dO, vw)
        dS = P * (dP - (P * dP).sum(axis=-1, keepdims=True))                # softmax Jacobian
        dqw = np.einsum("nhpq,nqhd->nphd", dS, kw)
        dkw = np.einsum("nhpq,nphd->nqhd", dS, qw)
        dSh = dS.sum(axis=0)                                                # [gh,N,N]
        for hh in range(gh):
            np.add.at(dtable[:, h0 + hh], rel.ravel(), dSh[hh].ravel())
        for dst, src, sl, wd in ((dq, dqw, chq, wq), (dk, dkw, chq, wq), (dv, dvw, ch, wv)):
            dst[..., sl] = reverse_shift(window_reverse(src.reshape(-1, N, gh * wd), M, B, H, W), s)
        h0 += gh
    dqkv = np.concatenate([dq * scale, dk, dv], axis=-1).reshape(-1, nh * (2 * wq + wv))
    dw_qkv = dqkv.T @ x.reshape(-1, C)
    db_qkv = dqkv.sum(axis=0)
    dx = (dqkv @ w_qkv).reshape(B, H, W, C)
    return dict(dx=dx, dw_qkv=dw_qkv, db_qkv=db_qkv, dw_proj=dw_proj, db_proj=db_proj, dbias_table=dtable)


def forward_backward_chunked(x, w_qkv, b_qkv, w_proj, b_proj, table, M, group_heads, group_shift, dy, chunk=4,
                             qk_dim=None, v_dim=None):
    """Same results as forward + backward, walking the batch `chunk` images at a time to bound memory."""
    B = x.shape[0]
    ys, dxs, acc = [], [], None
    for b0 in range(0, B, chunk):
        y, cache = forward(x[b0:b0 + chunk], w_qkv, b_qkv, w_proj, b_proj, table, M, group_heads, group_shift,
                           qk_dim=qk_dim, v_dim=v_dim)
        g = backward(cache, dy[b0:b0 + chunk])
        ys.append(y)
        dxs.append(g.pop("dx"))
        acc = g if acc is None else {n: acc[n] + g[n] for n in acc}
    acc["dx"] = np.concatenate(dxs, axis=0)
    return np.concatenate(ys, axis=0), acc


# --------------------------------------------------------------------------
# forward, brute force over the whole image (no roll, no partition, no region labels)
# --------------------------------------------------------------------------
def bruteforce_forward(x, w_qkv, b_qkv, w_proj, b_proj, table, M, group_heads, group_shift, qk_dim=None, v_dim=None):
    """Masked global attention in original coordinates; pure loops, tiny inputs only.

    A shifted group cuts the image at rows/cols s + k*M.  Two tokens may attend
    to one another iff floor((i - s)/M) agrees on both axes (floor toward
    -inf, so the strip [0,s) is its own segment).  Inside one segment slot
    offsets equal coordinate offsets, hence the bias row is taken from
    coordinate differences.
    """
    x = np.asarray(x, F64)
    w_qkv = np.asarray(w_qkv, F64)
    w_proj = np.asarray(w_proj, F64)
    table = np.asarray(table, F64)
    B, H, W, C, nh, d = _check(x, group_heads, group_shift, M)
    dq, dv = _widths(d, qk_dim, v_dim)
    Cq, Cv = nh * dq, nh * dv
    b_qkv = np.zeros(2 * Cq + Cv, F64) if b_qkv is None else np.asarray(b_qkv, F64)
    b_proj = np.zeros(C, F64) if b_proj is None else np.asarray(b_proj, F64)
    head_shift = [s for gh, s in zip(group_heads, group_shift) for _ in range(gh)]
    A = np.zeros((B, H, W, Cv), F64)
    for b in range(B):
        tok = x[b].reshape(H * W, C)
        for h in range(nh):
            s = head_shift[h]
            rq = slice(h * dq, (h + 1) * dq)
            rk = slice(Cq + h * dq, Cq + (h + 1) * dq)
            rv = slice(2 * Cq + h * dv, 2 * Cq + (h + 1) * dv)
            q = tok @ w_qkv[rq].T + b_qkv[rq]
            k = tok @ w_qkv[rk].T + b_qkv[rk]
            v = tok @ w_qkv[rv].T + b_qkv[rv]
            for p in range(H * W):
                ip, jp = divmod(p, W)
                logits, keys = [], []
                for r in range(H * W):
                    ir, jr = divmod(r, W)
                    if (ip - s) // M != (ir - s) // M or (jp - s) // M != (jr - s) // M:
                        continue
                    row = (ip - ir + M - 1) * (2 * M - 1) + (jp - jr + M - 1)
                    logits.append(float(q[p] @ k[r]) / np.sqrt(dq) + table[row, h])
                    keys.append(r)
                logits = np.array(logits)
                wgt = np.exp(logits - logits.max())
                wgt /= wgt.sum()
                A[b, ip, jp, h * dv:(h + 1) * dv] = wgt @ v[keys]
    return A @ w_proj.T + b_proj

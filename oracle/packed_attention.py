"""CPU oracle for packed (block-diagonal causal) attention -- TEST INFRASTRUCTURE.

Plain numpy, fp64, written from the method's definition; it shares no code with
the CUDA library and must only be used by the tests, the smoke check and the
CPU-baseline leg of the benchmark.  Every function is pinned by the CPU tests
(worked example of Sec. 3.5, brute force, closed forms, finite differences,
library cross-checks); nothing here is "parity unpinned".

Notation: a stream of T tokens holds E examples; example e occupies tokens
[s_e, s_{e+1}) and has length L_e.  Hq query heads, Hkv key/value heads,
G = Hq / Hkv, query head h reads kv head h // G.  D = head_dim.

What the method computes (Sec. 3 "Packing with Position IDs", Sec. 3.1, and the
paragraph after Table 1): example boundaries are read off ``position_ids``
(which restart at every example), ``cu_seq_len`` is built from them, and
attention is evaluated per example with a causal mask, so that no token sees
another example (Table 1, column "Correct Cross-Attention").
"""
from __future__ import annotations

import numpy as np

# ----------------------------------------------------------------------------
# boundaries (paragraph after Table 1: cu_seq_len from position_ids)
# ----------------------------------------------------------------------------


def seqlens_from_posids(position_ids):
    """Example starts from ``position_ids``.

    Token t starts an example iff t == 0 or pos[t] <= pos[t-1] (ids only grow
    inside an example and restart at a boundary, Sec. 3.1).  Returns
    ``(cu_seqlens int32 [T+1], n_examples, max_seqlen)``; ``cu_seqlens[:E+1]``
    are the start offsets followed by T, the remaining entries are T.
    """
    pos = np.asarray(position_ids, dtype=np.int64).reshape(-1)
    T = pos.shape[0]
    starts = []
    for t in range(T):
        if t == 0 or pos[t] <= pos[t - 1]:
            starts.append(t)
    E = len(starts)
    cu = np.full((T + 1,), T, dtype=np.int32)
    for e, s in enumerate(starts):
        cu[e] = s
    max_len = 0
    for e in range(E):
        max_len = max(max_len, int(cu[e + 1]) - int(cu[e]))
    return cu, E, max_len


def example_ids(position_ids):
    """Example index of every token (number of starts in [0, t] minus one)."""
    pos = np.asarray(position_ids, dtype=np.int64).reshape(-1)
    out = np.zeros(pos.shape[0], dtype=np.int64)
    e = -1
    for t in range(pos.shape[0]):
        if t == 0 or pos[t] <= pos[t - 1]:
            e += 1
        out[t] = e
    return out


# ----------------------------------------------------------------------------
# per-tile work lists
# ----------------------------------------------------------------------------


def work_lists(cu_seqlens, n_examples, bm, bn):
    """Tiles that hold at least one (query, key) pair of the block-diagonal
    causal mask, listed per example and block in ascending order.

    forward item  (q_start, q_len, kv_start, kv_len): a block of <= bm query
        rows of one example together with the key range it may see.
    backward item (kv_start, kv_len, q_start, q_len): a block of <= bn key rows
        of one example together with the query range that may see it.
    ``*_order`` is the stable sort of the item indices by descending tile count of the
    item's EXAMPLE (ceil(L_e / bm)): long examples first, the items of one example adjacent
    and in block order.  Both lists have the same order.
    """
    assert bm == bn, "the lists are defined for square tiles"
    fwd, bwd = [], []
    for e in range(n_examples):
        s, t = int(cu_seqlens[e]), int(cu_seqlens[e + 1])
        L = t - s
        b = 0
        while b * bm < L:
            q_len = min(bm, L - b * bm)
            fwd.append((s + b * bm, q_len, s, b * bm + q_len))
            b += 1
        b = 0
        while b * bn < L:
            kv_len = min(bn, L - b * bn)
            bwd.append((s + b * bn, kv_len, s + b * bn, t - (s + b * bn)))
            b += 1
    fwd = np.asarray(fwd, dtype=np.int32).reshape(-1, 4)
    bwd = np.asarray(bwd, dtype=np.int32).reshape(-1, 4)
    ex_tiles = []
    for e in range(n_examples):
        n = -(-(int(cu_seqlens[e + 1]) - int(cu_seqlens[e])) // bm)
        ex_tiles.extend([n] * n)
    order = sorted(range(len(fwd)), key=lambda i: -ex_tiles[i])      # sorted() is stable
    fwd_order = np.asarray(order, dtype=np.int32)
    bwd_order = np.asarray(order, dtype=np.int32)
    return fwd, bwd, fwd_order, bwd_order


# ----------------------------------------------------------------------------
# rotary embedding indexed by position_ids
# ----------------------------------------------------------------------------


def rope(x, position_ids, theta, inverse=False):
    """Rotate every (token, head) vector: pairs (i, i + D/2), angle
    pos * theta**(-2 i / D); ``inverse`` rotates by the negative angle."""
    x = np.asarray(x, dtype=np.float64)
    T, H, D = x.shape
    half = D // 2
    pos = np.asarray(position_ids, dtype=np.float64).reshape(T, 1, 1)
    i = np.arange(half, dtype=np.float64).reshape(1, 1, half)
    phi = pos * np.power(float(theta), -2.0 * i / D)
    if inverse:
        phi = -phi
    c, s = np.cos(phi), np.sin(phi)
    x1, x2 = x[..., :half], x[..., half:]
    out = np.empty_like(x)
    out[..., :half] = x1 * c - x2 * s
    out[..., half:] = x2 * c + x1 * s
    return out


# ----------------------------------------------------------------------------
# attention, one (example, query head) at a time
# ----------------------------------------------------------------------------

_ROW_BLOCK = 2048   # memory bound only: query rows are independent of each other


def _visible(rows, cols, window):
    """Causal mask of one example, optionally limited to the ``window`` most recent keys
    (the row's own position included); window <= 0 means no limit."""
    m = cols <= rows
    if window > 0:
        m = m & (cols > rows - window)
    return m


def _example_head_fwd(q, k, v, scale, window=0):
    """q [L, D], k/v [L, D] of ONE example and head -> (O [L, D], lse [L])."""
    L = q.shape[0]
    out = np.empty((L, v.shape[1]), dtype=np.float64)
    lse = np.empty((L,), dtype=np.float64)
    for r0 in range(0, L, _ROW_BLOCK):
        r1 = min(L, r0 + _ROW_BLOCK)
        s = scale * (q[r0:r1] @ k[:r1].T)                       # keys j <= i only
        rows = np.arange(r0, r1).reshape(-1, 1)
        cols = np.arange(0, r1).reshape(1, -1)
        s = np.where(_visible(rows, cols, window), s, -np.inf)   # causal, diagonal kept
        m = s.max(axis=1, keepdims=True)
        z = np.exp(s - m).sum(axis=1, keepdims=True)
        l = m + np.log(z)
        p = np.exp(s - l)
        out[r0:r1] = p @ v[:r1]
        lse[r0:r1] = l[:, 0]
    return out, lse


def _example_head_bwd(do, q, k, v, scale, window=0):
    """Gradients of ONE example and head w.r.t. its (already rotated) q, k and v."""
    L = q.shape[0]
    dq = np.zeros_like(q)
    dk = np.zeros_like(k)
    dv = np.zeros_like(v)
    for r0 in range(0, L, _ROW_BLOCK):
        r1 = min(L, r0 + _ROW_BLOCK)
        s = scale * (q[r0:r1] @ k[:r1].T)
        rows = np.arange(r0, r1).reshape(-1, 1)
        cols = np.arange(0, r1).reshape(1, -1)
        s = np.where(_visible(rows, cols, window), s, -np.inf)
        m = s.max(axis=1, keepdims=True)
        l = m + np.log(np.exp(s - m).sum(axis=1, keepdims=True))
        p = np.exp(s - l)                                        # masked entries are 0
        o = p @ v[:r1]
        delta = (do[r0:r1] * o).sum(axis=1, keepdims=True)      # row sum of dO * O
        dp = do[r0:r1] @ v[:r1].T
        ds = p * (dp - delta)
        dv[:r1] += p.T @ do[r0:r1]
        dq[r0:r1] = scale * (ds @ k[:r1])
        dk[:r1] += scale * (ds.T @ q[r0:r1])
    return dq, dk, dv


def _f64(x):
    return np.asarray(x, dtype=np.float64)


def attn_fwd(q, k, v, position_ids, softmax_scale, rope_theta=0.0, examples=None, window=0):
    """Forward over a packed stream.

    q [T, Hq, D], k/v [T, Hkv, D].  Returns (out fp64 [T, Hq, D], lse fp64
    [Hq, T]); lse is the natural log of the sum of exp(scale * q.k) over the
    keys the row may see.  ``examples`` restricts the work to those example
    indices (other rows are left as NaN).  ``window`` > 0 limits every row to its
    ``window`` most recent keys inside its example (sliding-window attention of
    the Mistral family; the row's own position counts).
    """
    q, k, v = _f64(q), _f64(k), _f64(v)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    cu, E, _ = seqlens_from_posids(position_ids)
    if rope_theta > 0:
        q = rope(q, position_ids, rope_theta)
        k = rope(k, position_ids, rope_theta)
    out = np.full((T, Hq, D), np.nan)
    lse = np.full((Hq, T), np.nan)
    todo = range(E) if examples is None else examples
    for e in todo:
        s, t = int(cu[e]), int(cu[e + 1])
        for h in range(Hq):
            g = h // G
            o, l = _example_head_fwd(q[s:t, h], k[s:t, g], v[s:t, g], softmax_scale, window)
            out[s:t, h] = o
            lse[h, s:t] = l
    return out, lse


def attn_bwd(dout, q, k, v, position_ids, softmax_scale, rope_theta=0.0, examples=None,
             window=0):
    """Backward over a packed stream: (dq [T,Hq,D], dk, dv [T,Hkv,D]) in fp64.

    dK and dV of a kv head are summed over the G query heads that read it.  With
    ``rope_theta > 0`` the gradients are with respect to the un-rotated q and k
    (the rotation is orthogonal, so its transpose is the inverse rotation).
    """
    dout, q, k, v = _f64(dout), _f64(q), _f64(k), _f64(v)
    T, Hq, D = q.shape
    Hkv = k.shape[1]
    G = Hq // Hkv
    cu, E, _ = seqlens_from_posids(position_ids)
    if rope_theta > 0:
        q = rope(q, position_ids, rope_theta)
        k = rope(k, position_ids, rope_theta)
    dq = np.full((T, Hq, D), np.nan)
    dk = np.full((T, Hkv, D), np.nan)
    dv = np.full((T, Hkv, D), np.nan)
    todo = range(E) if examples is None else examples
    for e in todo:
        s, t = int(cu[e]), int(cu[e + 1])
        dk[s:t] = 0.0
        dv[s:t] = 0.0
        for h in range(Hq):
            g = h // G
            a, b, c = _example_head_bwd(dout[s:t, h], q[s:t, h], k[s:t, g], v[s:t, g],
                                        softmax_scale, window)
            dq[s:t, h] = a
            dk[s:t, g] += b
            dv[s:t, g] += c
    if rope_theta > 0:
        dq = rope(dq, position_ids, rope_theta, inverse=True)
        dk = rope(dk, position_ids, rope_theta, inverse=True)
    return dq, dk, dv


def delta_rows(dout, out):
    """delta[h, i] = sum_d dO[i, h, d] * O[i, h, d] (the backward's row term)."""
    return (_f64(dout) * _f64(out)).sum(axis=2).T.copy()


# ----------------------------------------------------------------------------
# single rows, for spot checks at sizes where a full pass is too slow
# ----------------------------------------------------------------------------


def attn_fwd_row(q, k, v, position_ids, softmax_scale, rope_theta, i, h):
    """(O[i, h, :], lse[h, i]) of one token and query head, from the definition."""
    cu, E, _ = seqlens_from_posids(position_ids)
    eid = int(np.searchsorted(cu[:E + 1], i, side="right") - 1)
    s = int(cu[eid])
    Hq, Hkv = q.shape[1], k.shape[1]
    g = h // (Hq // Hkv)
    pos = np.asarray(position_ids)
    qi = _f64(q[i:i + 1, h:h + 1])
    kk = _f64(k[s:i + 1, g:g + 1])
    vv = _f64(v[s:i + 1, g])
    if rope_theta > 0:
        qi = rope(qi, pos[i:i + 1], rope_theta)
        kk = rope(kk, pos[s:i + 1], rope_theta)
    sc = softmax_scale * (kk[:, 0] @ qi[0, 0])
    m = sc.max()
    l = m + np.log(np.exp(sc - m).sum())
    p = np.exp(sc - l)
    return p @ vv, l


def attn_bwd_dq_row(dout, q, k, v, position_ids, softmax_scale, rope_theta, i, h):
    """dQ[i, h, :] of one token and query head, from the definition."""
    cu, E, _ = seqlens_from_posids(position_ids)
    eid = int(np.searchsorted(cu[:E + 1], i, side="right") - 1)
    s = int(cu[eid])
    Hq, Hkv = q.shape[1], k.shape[1]
    g = h // (Hq // Hkv)
    pos = np.asarray(position_ids)
    qi = _f64(q[i:i + 1, h:h + 1])
    kk = _f64(k[s:i + 1, g:g + 1])
    vv = _f64(v[s:i + 1, g])
    if rope_theta > 0:
        qi = rope(qi, pos[i:i + 1], rope_theta)
        kk = rope(kk, pos[s:i + 1], rope_theta)
    sc = softmax_scale * (kk[:, 0] @ qi[0, 0])
    m = sc.max()
    l = m + np.log(np.exp(sc - m).sum())
    p = np.exp(sc - l)
    o = p @ vv
    do = _f64(dout[i, h])
    delta = float(do @ o)
    dp = vv @ do
    ds = p * (dp - delta)
    dq = softmax_scale * (ds @ kk[:, 0])
    if rope_theta > 0:
        dq = rope(dq.reshape(1, 1, -1), pos[i:i + 1], rope_theta, inverse=True)[0, 0]
    return dq

"""Pins for the CPU oracle: every function is checked against something other
than itself -- the paper's worked example, brute force over a dense mask,
closed forms, finite differences and library routines (torch SDPA / autograd in
fp64 on CPU, used as a second opinion only)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, vals = line.split(":")
            out[key.strip()] = [int(x) for x in vals.split()]
    return out


# ---------------------------------------------------------------- boundaries

def test_worked_example_sec3_5():
    g = _read_golden("worked_example_sec3_5.txt")
    cu, E, mx = orc.seqlens_from_posids(g["position_ids"])
    assert E == 4 and mx == 11
    assert cu[:5].tolist() == g["cu_seqlens"] == [0, 4, 12, 17, 28]
    assert (cu[5:] == 28).all() and cu.shape[0] == 29
    # the -100 labels of the paper sit exactly on the recovered starts
    starts = [i for i, l in enumerate(g["labels"]) if l == -100]
    assert starts == cu[:4].tolist()


@pytest.mark.parametrize("seed", range(8))
def test_roundtrip_lengths(seed):
    rng = np.random.default_rng(seed)
    lens = [int(x) for x in rng.integers(1, 40, size=rng.integers(1, 30))]
    pos = wl.position_ids_from_lengths(lens)
    cu, E, mx = orc.seqlens_from_posids(pos)
    assert E == len(lens) and mx == max(lens)
    assert np.diff(cu[:E + 1]).tolist() == lens


def test_reset_rules_agree_on_configs():
    for name in wl.WORKLOAD_NAMES:
        w = wl.workload(name)
        for lens in w.streams[:4]:
            pos = wl.position_ids_from_lengths(lens).astype(np.int64)
            cu, E, _ = orc.seqlens_from_posids(pos)
            by_zero = np.flatnonzero(pos == 0)
            by_step = np.flatnonzero(np.concatenate([[True], pos[1:] != pos[:-1] + 1]))
            assert cu[:E].tolist() == by_zero.tolist() == by_step.tolist()


def test_reset_rule_special_cases():
    # fragment opening a pack keeps its ids, token 0 still starts an example
    cu, E, mx = orc.seqlens_from_posids([5, 6, 7, 3, 4])
    assert (E, mx, cu[:3].tolist()) == (2, 3, [0, 3, 5])
    # strided ids stay together
    cu, E, mx = orc.seqlens_from_posids([0, 2, 4])
    assert (E, mx) == (1, 3)
    # repeated id is a restart
    cu, E, _ = orc.seqlens_from_posids([0, 0, 0])
    assert E == 3
    cu, E, mx = orc.seqlens_from_posids([])
    assert (E, mx, cu.tolist()) == (0, 0, [0])
    assert orc.example_ids([0, 1, 0, 0, 1, 2]).tolist() == [0, 0, 1, 2, 2, 2]


# ---------------------------------------------------------------- work lists

def _dense_mask(pos):
    eid = orc.example_ids(pos)
    T = len(pos)
    i = np.arange(T).reshape(-1, 1)
    j = np.arange(T).reshape(1, -1)
    return (eid.reshape(-1, 1) == eid.reshape(1, -1)) & (j <= i)


@pytest.mark.parametrize("bm,bn,lens", [
    (4, 4, [1, 3, 4, 5, 9, 2]), (4, 4, [17]), (8, 8, [7, 8, 9, 1, 1, 16]),
    (4, 4, [4, 4, 4]), (128, 128, [127, 128, 129, 1, 300])])
def test_work_lists_cover_exactly_the_mask(bm, bn, lens):
    pos = wl.position_ids_from_lengths(lens)
    T = len(pos)
    mask = _dense_mask(pos)
    cu, E, _ = orc.seqlens_from_posids(pos)
    fwd, bwd, fo, bo = orc.work_lists(cu, E, bm, bn)

    # forward: every item's (row block x key tiles) region; pairs covered once
    cover = np.zeros((T, T), dtype=np.int32)
    for qs, ql, ks, kl in fwd:
        ntile = -(-kl // bn)
        for t in range(ntile):
            c0, c1 = ks + t * bn, min(ks + (t + 1) * bn, T)
            # the tile must hold at least one valid pair (never scheduled otherwise)
            assert mask[qs:qs + ql, c0:c1].any()
            cover[qs:qs + ql, c0:min(c1, ks + kl)] += 1
    assert (cover[mask] == 1).all()
    # rows of an item belong to one example and its keys start at the example start
    eid = orc.example_ids(pos)
    for qs, ql, ks, kl in fwd:
        assert len(set(eid[qs:qs + ql])) == 1 and eid[ks] == eid[qs]
        assert ks == cu[eid[qs]] and ks + kl == qs + ql
    # backward: transpose view
    cover = np.zeros((T, T), dtype=np.int32)
    for ks, kl, qs, ql in bwd:
        assert qs == ks and eid[ks] == eid[qs + ql - 1]
        assert qs + ql == cu[eid[ks] + 1]
        cover[qs:qs + ql, ks:ks + kl] += 1
    assert (cover[mask] == 1).all()
    # closed forms for the counts
    assert len(fwd) == sum(-(-l // bm) for l in lens)
    assert len(bwd) == sum(-(-l // bn) for l in lens)
    # order: a permutation; examples by descending tile count (ties in stream order), the items
    # of an example adjacent and in block order
    ex_of = [int(eid[x[0]]) for x in fwd]
    ex_tiles = [sum(1 for y in ex_of if y == e) for e in ex_of]
    assert sorted(fo.tolist()) == list(range(len(fwd))) and fo.tolist() == bo.tolist()
    keys = [(-ex_tiles[i], i) for i in fo]
    assert keys == sorted(keys)
    for a, b in zip(fo[:-1], fo[1:]):
        if ex_of[a] == ex_of[b]:
            assert b == a + 1


def test_work_list_visit_counts_match_closed_form():
    # number of (q block, kv tile) visits of the 128x128 tiling, all five configs
    expect = {"c1": 10, "c2": 849, "c3": 20312, "c4": 21600, "c5": 21293}
    for name, n in expect.items():
        w = wl.workload(name)
        tot = 0
        for lens in w.streams:
            pos = wl.position_ids_from_lengths(lens)
            cu, E, _ = orc.seqlens_from_posids(pos)
            fwd, bwd, _, _ = orc.work_lists(cu, E, 128, 128)
            tot += sum(-(-int(x[3]) // 128) for x in fwd)
            closed = sum(sum(-(-min((b + 1) * 128, l) // 128) for b in range(-(-l // 128)))
                         for l in lens)
            assert sum(-(-int(x[3]) // 128) for x in fwd) == closed
            assert sum(-(-int(x[3]) // 128) for x in bwd) == closed
        assert tot == n


# ---------------------------------------------------------------- rope

def test_rope_closed_forms():
    # D = 2: one pair, frequency 1 -> plain rotation by pos radians
    x = np.array([[[1.0, 0.0]], [[0.0, 2.0]]])
    y = orc.rope(x, [1, 3], 1e4)
    assert np.allclose(y[0, 0], [math.cos(1), math.sin(1)], atol=1e-15)
    assert np.allclose(y[1, 0], [-2 * math.sin(3), 2 * math.cos(3)], atol=1e-15)
    # D = 4, theta = 1e4: second pair has frequency 1e4**(-2/4) = 0.01
    x = np.array([[[0.0, 1.0, 0.0, 0.0]]])
    y = orc.rope(x, [100], 1e4)
    assert np.allclose(y[0, 0], [0.0, math.cos(1.0), 0.0, math.sin(1.0)], atol=1e-13)
    # pairing is (i, i + D/2), not (2i, 2i+1)
    x = np.array([[[1.0, 0.0, 0.0, 0.0]]])
    y = orc.rope(x, [2], 1e4)
    assert np.allclose(y[0, 0], [math.cos(2.0), 0.0, math.sin(2.0), 0.0], atol=1e-13)


def test_rope_properties():
    rng = np.random.default_rng(0)
    x = rng.standard_normal((9, 3, 16))
    pos = np.array([0, 1, 2, 3, 0, 1, 0, 7, 8])
    y = orc.rope(x, pos, 5e5)
    assert np.array_equal(y[pos == 0], x[pos == 0])
    assert np.allclose(np.linalg.norm(y, axis=2), np.linalg.norm(x, axis=2), rtol=1e-13)
    assert np.allclose(orc.rope(y, pos, 5e5, inverse=True), x, atol=1e-13)
    # rotations compose additively in the position
    assert np.allclose(orc.rope(orc.rope(x, pos, 5e5), 2 * pos, 5e5), orc.rope(x, 3 * pos, 5e5),
                       atol=1e-12)


def test_rope_relative_position_property():
    rng = np.random.default_rng(1)
    T, H, D = 12, 2, 8
    q, k, v = (rng.standard_normal((T, H, D)) for _ in range(3))
    pos = np.arange(T)
    o0, l0 = orc.attn_fwd(q, k, v, pos, 0.3, 1e4)
    o1, l1 = orc.attn_fwd(q, k, v, pos + 37, 0.3, 1e4)
    assert np.allclose(o0, o1, atol=1e-9) and np.allclose(l0, l1, atol=1e-9)


# ---------------------------------------------------------------- forward

def _brute_forward(q, k, v, pos, scale, G):
    """Scalar loops over the dense T x T mask; nothing shared with the oracle."""
    T, Hq, D = q.shape
    mask = _dense_mask(pos)
    out = np.zeros((T, Hq, D))
    lse = np.zeros((Hq, T))
    for h in range(Hq):
        g = h // G
        for i in range(T):
            w = []
            for j in range(T):
                if mask[i, j]:
                    w.append((j, math.exp(scale * sum(q[i, h, d] * k[j, g, d] for d in range(D)))))
            z = sum(x for _, x in w)
            lse[h, i] = math.log(z)
            for j, x in w:
                for d in range(D):
                    out[i, h, d] += x / z * v[j, g, d]
    return out, lse


def test_forward_brute_force_gqa():
    rng = np.random.default_rng(2)
    lens = [3, 1, 5, 2]
    T, Hq, Hkv, D = sum(lens), 4, 2, 4
    q = rng.standard_normal((T, Hq, D))
    k = rng.standard_normal((T, Hkv, D))
    v = rng.standard_normal((T, Hkv, D))
    pos = wl.position_ids_from_lengths(lens)
    o, l = orc.attn_fwd(q, k, v, pos, 0.7)
    ob, lb = _brute_forward(q, k, v, pos, 0.7, Hq // Hkv)
    assert np.allclose(o, ob, atol=1e-12) and np.allclose(l, lb, atol=1e-12)


def test_forward_brute_force_with_rope():
    rng = np.random.default_rng(3)
    lens = [4, 3]
    T, H, D = sum(lens), 2, 4
    q, k, v = (rng.standard_normal((T, H, D)) for _ in range(3))
    pos = wl.position_ids_from_lengths(lens)
    o, l = orc.attn_fwd(q, k, v, pos, 0.5, 1e4)
    ob, lb = _brute_forward(orc.rope(q, pos, 1e4), orc.rope(k, pos, 1e4), v, pos, 0.5, 1)
    assert np.allclose(o, ob, atol=1e-12) and np.allclose(l, lb, atol=1e-12)


def _sdpa(q, k, v, scale, mask=None, causal=False):
    """torch SDPA in fp64 on CPU: q [T,H,D] -> [T,H,D] (kv heads already expanded)."""
    tq, tk, tv = (torch.from_numpy(np.ascontiguousarray(x)).permute(1, 0, 2)[None] for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(
        tq, tk, tv, attn_mask=None if mask is None else torch.from_numpy(mask),
        is_causal=causal, scale=scale)
    return o[0].permute(1, 0, 2).numpy()


def test_single_example_is_plain_causal_attention():
    rng = np.random.default_rng(4)
    T, H, D = 33, 3, 8
    q, k, v = (rng.standard_normal((T, H, D)) for _ in range(3))
    o, _ = orc.attn_fwd(q, k, v, np.arange(T), 0.35)
    assert np.allclose(o, _sdpa(q, k, v, 0.35, causal=True), atol=1e-12)
    # and with two examples the result differs from plain causal (Table 1, packing w/o PosID)
    o2, _ = orc.attn_fwd(q, k, v, wl.position_ids_from_lengths([20, 13]), 0.35)
    assert np.abs(o2[20:] - o[20:]).max() > 1e-3
    assert np.allclose(o2[:20], o[:20], atol=1e-12)


def test_packed_equals_each_example_alone_and_padded():
    rng = np.random.default_rng(5)
    lens = [5, 9, 1, 7]
    T, Hq, Hkv, D = sum(lens), 4, 2, 8
    q = rng.standard_normal((T, Hq, D))
    k = rng.standard_normal((T, Hkv, D))
    v = rng.standard_normal((T, Hkv, D))
    do = rng.standard_normal((T, Hq, D))
    pos = wl.position_ids_from_lengths(lens)
    o, l = orc.attn_fwd(q, k, v, pos, 0.4, 1e4)
    dq, dk, dv = orc.attn_bwd(do, q, k, v, pos, 0.4, 1e4)
    s = 0
    Lmax = max(lens)
    for L in lens:
        sl = slice(s, s + L)
        # invariant 1: the example run alone
        oe, le = orc.attn_fwd(q[sl], k[sl], v[sl], np.arange(L), 0.4, 1e4)
        assert np.allclose(o[sl], oe, atol=1e-12) and np.allclose(l[:, sl], le, atol=1e-12)
        ge = orc.attn_bwd(do[sl], q[sl], k[sl], v[sl], np.arange(L), 0.4, 1e4)
        for a, b in zip((dq[sl], dk[sl], dv[sl]), ge):
            assert np.allclose(a, b, atol=1e-11)
        # invariant 3: right-padded to Lmax with random pad values, zero dO on pads
        pad = Lmax - L
        qp = np.concatenate([q[sl], rng.standard_normal((pad, Hq, D))])
        kp = np.concatenate([k[sl], rng.standard_normal((pad, Hkv, D))])
        vp = np.concatenate([v[sl], rng.standard_normal((pad, Hkv, D))])
        dop = np.concatenate([do[sl], np.zeros((pad, Hq, D))])
        op, lp = orc.attn_fwd(qp, kp, vp, np.arange(Lmax), 0.4, 1e4)
        assert np.allclose(op[:L], oe, atol=1e-12)
        gp = orc.attn_bwd(dop, qp, kp, vp, np.arange(Lmax), 0.4, 1e4)
        for a, b in zip(gp, ge):
            assert np.allclose(a[:L], b, atol=1e-11)
        s += L


def test_forward_closed_forms():
    rng = np.random.default_rng(6)
    lens = [6, 4]
    T, H, D = sum(lens), 2, 4
    q, k, v = (rng.standard_normal((T, H, D)) for _ in range(3))
    pos = wl.position_ids_from_lengths(lens)
    scale = 0.9
    o, l = orc.attn_fwd(q, k, v, pos, scale)
    for s in (0, 6):          # first token of an example sees only itself
        assert np.allclose(o[s], v[s], atol=1e-14)
        assert np.allclose(l[:, s], scale * (q[s] * k[s]).sum(-1), atol=1e-14)
    # all keys of an example equal -> running mean of v, lse = s + log(i + 1)
    k2 = k.copy()
    k2[:6] = k[0]
    o2, l2 = orc.attn_fwd(q, k2, v, pos, scale)
    for i in range(6):
        assert np.allclose(o2[i], v[:i + 1].mean(axis=0), atol=1e-13)
        assert np.allclose(l2[:, i], scale * (q[i] * k[0]).sum(-1) + math.log(i + 1), atol=1e-13)
    # V constant -> O constant
    v3 = np.ones_like(v) * 2.5
    o3, _ = orc.attn_fwd(q, k, v3, pos, scale)
    assert np.allclose(o3, 2.5, atol=1e-14)


def test_row_functions_match_full_pass():
    rng = np.random.default_rng(7)
    lens = [7, 5, 9]
    T, Hq, Hkv, D = sum(lens), 4, 2, 8
    q = rng.standard_normal((T, Hq, D))
    k = rng.standard_normal((T, Hkv, D))
    v = rng.standard_normal((T, Hkv, D))
    do = rng.standard_normal((T, Hq, D))
    pos = wl.position_ids_from_lengths(lens)
    for theta in (0.0, 1e4):
        o, l = orc.attn_fwd(q, k, v, pos, 0.3, theta)
        dq, _, _ = orc.attn_bwd(do, q, k, v, pos, 0.3, theta)
        for i, h in [(0, 0), (6, 3), (7, 1), (20, 2), (11, 0)]:
            oi, li = orc.attn_fwd_row(q, k, v, pos, 0.3, theta, i, h)
            assert np.allclose(oi, o[i, h], atol=1e-12) and abs(li - l[h, i]) < 1e-12
            assert np.allclose(orc.attn_bwd_dq_row(do, q, k, v, pos, 0.3, theta, i, h), dq[i, h],
                               atol=1e-12)


# ---------------------------------------------------------------- backward

def _loss(q, k, v, do, pos, scale, theta):
    o, _ = orc.attn_fwd(q, k, v, pos, scale, theta)
    return float((o * do).sum())


@pytest.mark.parametrize("theta", [0.0, 1e4])
def test_backward_finite_differences(theta):
    rng = np.random.default_rng(8)
    lens = [4, 6, 1]
    T, Hq, Hkv, D = sum(lens), 4, 2, 8
    q = rng.standard_normal((T, Hq, D))
    k = rng.standard_normal((T, Hkv, D))
    v = rng.standard_normal((T, Hkv, D))
    do = rng.standard_normal((T, Hq, D))
    pos = wl.position_ids_from_lengths(lens)
    scale = 0.45
    dq, dk, dv = orc.attn_bwd(do, q, k, v, pos, scale, theta)
    eps = 1e-6
    for name, x, g in (("q", q, dq), ("k", k, dk), ("v", v, dv)):
        for _ in range(25):
            idx = tuple(rng.integers(0, n) for n in x.shape)
            old = x[idx]
            x[idx] = old + eps
            lp = _loss(q, k, v, do, pos, scale, theta)
            x[idx] = old - eps
            lm = _loss(q, k, v, do, pos, scale, theta)
            x[idx] = old
            fd = (lp - lm) / (2 * eps)
            assert abs(fd - g[idx]) < 1e-7 * max(1.0, abs(fd)), (name, idx, fd, g[idx])


def test_backward_matches_torch_autograd():
    rng = np.random.default_rng(9)
    lens = [6, 3, 8]
    T, Hq, Hkv, D = sum(lens), 4, 2, 8
    G = Hq // Hkv
    q = rng.standard_normal((T, Hq, D))
    k = rng.standard_normal((T, Hkv, D))
    v = rng.standard_normal((T, Hkv, D))
    do = rng.standard_normal((T, Hq, D))
    pos = wl.position_ids_from_lengths(lens)
    tq, tk, tv = (torch.from_numpy(x).clone().requires_grad_(True) for x in (q, k, v))
    mask = torch.from_numpy(_dense_mask(pos))
    ke = tk.repeat_interleave(G, dim=1)
    ve = tv.repeat_interleave(G, dim=1)
    o = torch.nn.functional.scaled_dot_product_attention(
        tq.permute(1, 0, 2)[None], ke.permute(1, 0, 2)[None], ve.permute(1, 0, 2)[None],
        attn_mask=mask, scale=0.6)[0].permute(1, 0, 2)
    (o * torch.from_numpy(do)).sum().backward()
    oo, _ = orc.attn_fwd(q, k, v, pos, 0.6)
    assert np.allclose(oo, o.detach().numpy(), atol=1e-12)
    dq, dk, dv = orc.attn_bwd(do, q, k, v, pos, 0.6)
    assert np.allclose(dq, tq.grad.numpy(), atol=1e-11)
    assert np.allclose(dk, tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv, tv.grad.numpy(), atol=1e-11)


def test_backward_special_cases():
    rng = np.random.default_rng(10)
    lens = [5, 4]
    T, H, D = sum(lens), 2, 4
    k, v, do = (rng.standard_normal((T, H, D)) for _ in range(3))
    pos = wl.position_ids_from_lengths(lens)
    # q = 0 -> uniform P, dK = 0 and dV[j] = sum_i dO_i / (i + 1)
    q = np.zeros((T, H, D))
    dq, dk, dv = orc.attn_bwd(do, q, k, v, pos, 0.5)
    assert np.allclose(dk, 0.0, atol=1e-14)
    exp_dv = np.zeros_like(v)
    for s, L in ((0, 5), (5, 4)):
        for j in range(L):
            for i in range(j, L):
                exp_dv[s + j] += do[s + i] / (i + 1)
    assert np.allclose(dv, exp_dv, atol=1e-13)
    # delta helper
    o, _ = orc.attn_fwd(q, k, v, pos, 0.5)
    d = orc.delta_rows(do, o)
    assert d.shape == (H, T) and np.allclose(d[1, 3], (do[3, 1] * o[3, 1]).sum())
    # dV rows of an example depend on that example only (exactly, in fp64)
    q = rng.standard_normal((T, H, D))
    g0 = orc.attn_bwd(do, q, k, v, pos, 0.5)
    q2, k2, v2, do2 = q.copy(), k.copy(), v.copy(), do.copy()
    for x in (q2, k2, v2, do2):
        x[5:] *= -3.0
    g1 = orc.attn_bwd(do2, q2, k2, v2, pos, 0.5)
    for a, b in zip(g0, g1):
        assert np.array_equal(a[:5], b[:5])


def test_examples_subset_argument():
    rng = np.random.default_rng(11)
    lens = [5, 4, 6]
    T, H, D = sum(lens), 2, 4
    q, k, v, do = (rng.standard_normal((T, H, D)) for _ in range(4))
    pos = wl.position_ids_from_lengths(lens)
    o, l = orc.attn_fwd(q, k, v, pos, 0.5)
    o1, l1 = orc.attn_fwd(q, k, v, pos, 0.5, examples=[1])
    assert np.array_equal(o1[5:9], o[5:9]) and np.isnan(o1[:5]).all() and np.isnan(o1[9:]).all()
    g = orc.attn_bwd(do, q, k, v, pos, 0.5)
    g1 = orc.attn_bwd(do, q, k, v, pos, 0.5, examples=[2])
    for a, b in zip(g, g1):
        assert np.array_equal(a[9:], b[9:]) and np.isnan(b[:9]).all()


# ---------------------------------------------------------------- sliding window

def _dense_window_mask(pos, window):
    """Dense mask written out by hand: same example, key not after the query, and (window > 0)
    at most window - 1 positions before it."""
    pos = np.asarray(pos)
    T = len(pos)
    ex = np.zeros(T, dtype=np.int64)
    for t in range(1, T):
        ex[t] = ex[t - 1] + (1 if pos[t] <= pos[t - 1] else 0)
    m = np.zeros((T, T), dtype=bool)
    for i in range(T):
        for j in range(T):
            m[i, j] = ex[i] == ex[j] and j <= i and (window <= 0 or i - j < window)
    return m


@pytest.mark.parametrize("window", [1, 2, 3, 5, 100])
def test_sliding_window_against_torch_sdpa_and_autograd(window):
    rng = np.random.default_rng(20 + window)
    lens = [7, 1, 9, 4]
    T, Hq, Hkv, D = sum(lens), 4, 2, 8
    G = Hq // Hkv
    q = rng.standard_normal((T, Hq, D))
    k = rng.standard_normal((T, Hkv, D))
    v = rng.standard_normal((T, Hkv, D))
    do = rng.standard_normal((T, Hq, D))
    pos = wl.position_ids_from_lengths(lens)
    mask = _dense_window_mask(pos, window)
    tq, tk, tv = (torch.from_numpy(x).clone().requires_grad_(True) for x in (q, k, v))
    o = torch.nn.functional.scaled_dot_product_attention(
        tq.permute(1, 0, 2)[None], tk.repeat_interleave(G, dim=1).permute(1, 0, 2)[None],
        tv.repeat_interleave(G, dim=1).permute(1, 0, 2)[None], attn_mask=torch.from_numpy(mask),
        scale=0.6)[0].permute(1, 0, 2)
    (o * torch.from_numpy(do)).sum().backward()
    oo, ll = orc.attn_fwd(q, k, v, pos, 0.6, window=window)
    assert np.allclose(oo, o.detach().numpy(), atol=1e-12)
    dq, dk, dv = orc.attn_bwd(do, q, k, v, pos, 0.6, window=window)
    assert np.allclose(dq, tq.grad.numpy(), atol=1e-11)
    assert np.allclose(dk, tk.grad.numpy(), atol=1e-11)
    assert np.allclose(dv, tv.grad.numpy(), atol=1e-11)
    # the row sees min(window, position + 1) keys: lse of all-zero scores would be its log
    z, lz = orc.attn_fwd(np.zeros_like(q), k, v, pos, 0.6, window=window)
    seen = np.minimum(window, np.asarray(pos) + 1)
    assert np.allclose(lz, np.log(seen)[None, :].repeat(Hq, 0), atol=1e-12)


def test_sliding_window_special_cases():
    rng = np.random.default_rng(30)
    lens = [6, 10]
    T, H, D = sum(lens), 2, 4
    q, k, v = (rng.standard_normal((T, H, D)) for _ in range(3))
    pos = wl.position_ids_from_lengths(lens)
    # window 1: every row sees itself only -> out = v, lse = its own score
    o, l = orc.attn_fwd(q, k, v, pos, 0.5, window=1)
    assert np.allclose(o, v, atol=1e-14)
    assert np.allclose(l, 0.5 * np.einsum("thd,thd->ht", q, k), atol=1e-13)
    # a window at least as long as the longest example changes nothing; 0 means no window
    a, la = orc.attn_fwd(q, k, v, pos, 0.5)
    for wdw in (10, 11, 1000, 0):
        b, lb = orc.attn_fwd(q, k, v, pos, 0.5, window=wdw)
        assert np.array_equal(a, b) and np.array_equal(la, lb)
    # with rope: the window is over positions inside the example, like the mask
    c, _ = orc.attn_fwd(q, k, v, pos, 0.5, 1e4, window=3)
    d, _ = orc.attn_fwd(orc.rope(q, pos, 1e4), orc.rope(k, pos, 1e4), v, pos, 0.5, window=3)
    assert np.allclose(c, d, atol=1e-13)

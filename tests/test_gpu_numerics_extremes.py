"""Parity with the fp64 oracle on inputs that stress the online softmax: near one-hot and near
uniform rows, a running maximum that grows at every key tile or never after the first, and the
closed forms (q = 0: running mean of v).  Tolerances as everywhere (O, lse 1e-2, gradients 2e-2
on fp32 outputs) except for the rows close to one-hot, where the bound is derived in the test."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import workloads as wl
from helpers import f64, max_abs, run_bwd, run_fwd, to_cuda

pytestmark = pytest.mark.gpu


def _check(st, w, theta=0.0, tol_o=1e-2, tol_g=2e-2, grad_rel=0.0):
    pos = st.position_ids.cpu().numpy()
    out, lse, ws = run_fwd(st, w, theta=theta)
    o_ref, l_ref = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta)
    assert np.isfinite(f64(out)).all() and np.isfinite(f64(lse)).all()
    assert max_abs(f64(out), o_ref) <= tol_o
    # lse grows with the logits: the bound is relative to its size beyond 1
    assert (np.abs(f64(lse) - l_ref) <= 1e-2 * np.maximum(1.0, np.abs(l_ref) / 16)).all()
    grads = run_bwd(st, w, out, lse, ws, theta=theta)
    refs = orc.attn_bwd(f64(st.dout), f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta)
    for name, g, e in zip(("dq", "dk", "dv"), grads, refs):
        assert np.isfinite(f64(g)).all(), name
        bound = max(tol_g, grad_rel * np.abs(e).max())
        assert max_abs(f64(g), e) <= bound, (name, max_abs(f64(g), e), bound)
    return out, lse


def _tensors(lens, Hq, Hkv, D, seed):
    w = wl.Workload("t", seed, Hq, Hkv, D, 0.0, [lens], "test")
    return w, to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))


@pytest.mark.parametrize("gain", [4.0, 0.01])
def test_peaked_and_flat_rows(gain):
    # logits of standard deviation 16 (rows close to one-hot) and 1e-4 (rows close to uniform)
    w, st = _tensors([700, 129, 60], 4, 2, 128, 70)
    st.q.mul_(gain)
    st.k.mul_(gain)
    if gain < 1:
        _check(st, w)
    else:
        # With a few keys carrying a row, the bf16 rounding of P and dS (2^-9 relative each) no
        # longer averages out over many keys: O is off by up to 2^-9 max|v| from P and as much again
        # from the row sum taken before the rounding; the gradients carry the same relative error
        # times the 4x larger q / k through their contraction: 2^-7 of the largest entry.
        _check(st, w, tol_o=2.0 ** -8 * float(st.v.float().abs().max()), grad_rel=2.0 ** -7)


def test_running_maximum_grows_at_every_key_tile():
    # k_j = (j / L) u, q_i = c u: the score of key j grows with j, so every new key tile raises the
    # row maximum and the accumulated output is rescaled at every step
    lens = [1100]
    w, st = _tensors(lens, 2, 2, 128, 71)
    g = torch.Generator().manual_seed(72)
    u = torch.randn(128, generator=g)
    u = (u / u.norm()).cuda()
    ramp = (torch.arange(lens[0], device="cuda", dtype=torch.float32) / lens[0])[:, None, None]
    st.k.copy_((ramp * u * 60.0).to(torch.bfloat16).expand_as(st.k))
    st.q.copy_((u * 8.0).to(torch.bfloat16).expand_as(st.q))
    _check(st, w)


def test_first_key_dominates_every_row():
    # an attention sink: key 0 of each example scores far above the rest, so the maximum is set in
    # the first key tile and never changes
    lens = [600, 300]
    w, st = _tensors(lens, 4, 1, 128, 73)
    starts = [0, 600]
    for s in starts:
        st.k[s] = st.q[s:s + 1].float().mean(dim=(0, 1)).to(torch.bfloat16) * 0 + 3.0
    st.q.copy_(st.q.abs())
    _check(st, w)


def test_zero_queries_give_the_running_mean_of_v():
    lens = [300, 77]
    w, st = _tensors(lens, 4, 2, 64, 74)
    st.q.zero_()
    out, lse = _check(st, w)
    v = f64(st.v)
    o = f64(out)
    s = 0
    for n in lens:
        mean = np.cumsum(v[s:s + n], axis=0) / np.arange(1, n + 1)[:, None, None]
        assert max_abs(o[s:s + n], np.repeat(mean, 2, axis=1)) <= 1e-2
        assert max_abs(f64(lse)[:, s:s + n], np.log(np.arange(1, n + 1))[None, :].repeat(4, 0)) <= 1e-2
        s += n

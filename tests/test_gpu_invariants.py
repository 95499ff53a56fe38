"""Invariants of the packed path on the GPU.

(1) Rows of O, lse, dV and dK of an example are BITWISE unchanged when finite values of other
    examples are perturbed (the schedule depends on position_ids only, masked probabilities are
    exactly zero, dK/dV accumulate in a fixed order); dQ is held to the tolerance.
(2) Packed == each example alone; single example == plain causal; padded == packed on non-pad
    rows (Table 1, "Correct Cross-Attention"); with two examples the result differs from plain
    causal attention over the whole stream.
(3) One flat stream of several packs is bit-identical to one call per pack.
(4) Two runs of the same call give bitwise equal O, lse, dK, dV."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from paper_2407_09105_b200 import api, workloads as wl
from helpers import f64, max_abs, run_bwd, run_fwd, to_cuda

pytestmark = pytest.mark.gpu


def _run(st, w, theta=None):
    out, lse, ws = run_fwd(st, w, torch.float32, theta=theta)
    dq, dk, dv = run_bwd(st, w, out, lse, ws, torch.float32, theta=theta)
    return out, lse, dq, dk, dv


@pytest.mark.parametrize("theta", [0.0, 1e4])
def test_other_examples_do_not_leak(theta):
    """(rotated-copies mode; with theta > 0 dQ is bitwise stable there as well)"""
    lens = [200, 130, 77, 300]
    w = wl.Workload("t", 21, 8, 2, 128, theta, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0))
    base = _run(st, w)
    s, e = 200, 330                                   # example 1 is kept, all others perturbed
    keep = torch.zeros(sum(lens), dtype=torch.bool, device="cuda")
    keep[s:e] = True
    g = torch.Generator(device="cuda").manual_seed(5)
    st2 = wl.StreamTensors(st.position_ids, st.q.clone(), st.k.clone(), st.v.clone(),
                           st.dout.clone(), lens)
    for x in (st2.q, st2.k, st2.v, st2.dout):
        noise = (torch.randn(x.shape, generator=g, device="cuda") * 50.0).to(torch.bfloat16)
        x[~keep] = -3.0 * x[~keep] + noise[~keep]
    pert = _run(st2, w)
    out0, lse0, dq0, dk0, dv0 = base
    out1, lse1, dq1, dk1, dv1 = pert
    assert torch.equal(out0[s:e], out1[s:e]) and torch.equal(lse0[:, s:e], lse1[:, s:e])
    assert torch.equal(dv0[s:e], dv1[s:e]) and torch.equal(dk0[s:e], dk1[s:e])
    assert max_abs(f64(dq0[s:e]), f64(dq1[s:e])) <= 2e-2
    assert not torch.equal(out0[:s], out1[:s])


def test_packed_equals_alone_and_padded_and_differs_from_plain_causal():
    lens = [150, 260, 40]
    Hq, Hkv, D = 4, 2, 128
    w = wl.Workload("t", 22, Hq, Hkv, D, 1e4, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0))
    out, lse, dq, dk, dv = _run(st, w)
    Lmax = max(lens)
    s = 0
    for L in lens:
        sl = slice(s, s + L)
        one = wl.StreamTensors(st.position_ids[sl].contiguous(), st.q[sl].contiguous(),
                               st.k[sl].contiguous(), st.v[sl].contiguous(),
                               st.dout[sl].contiguous(), [L])
        o1, l1, dq1, dk1, dv1 = _run(one, w)
        # same tiles, same order: the example alone is bit-identical to its rows in the pack
        assert torch.equal(o1, out[sl]) and torch.equal(l1, lse[:, sl])
        assert torch.equal(dk1, dk[sl]) and torch.equal(dv1, dv[sl])
        assert max_abs(f64(dq1), f64(dq[sl])) <= 1e-3
        # right-padded row of length Lmax (pad tokens random, their dO zero)
        pad = Lmax - L
        g = torch.Generator(device="cuda").manual_seed(L)
        mk = lambda x: torch.cat([x[sl], torch.randn((pad,) + x.shape[1:], generator=g,
                                                     device="cuda").to(torch.bfloat16)])
        padded = wl.StreamTensors(torch.arange(Lmax, dtype=torch.int32, device="cuda"),
                                  mk(st.q), mk(st.k), mk(st.v),
                                  torch.cat([st.dout[sl], torch.zeros((pad, Hq, D), device="cuda",
                                                                      dtype=torch.bfloat16)]), [Lmax])
        o2, l2, dq2, dk2, dv2 = _run(padded, w)
        assert torch.equal(o2[:L], out[sl]) and torch.equal(l2[:, :L], lse[:, sl])
        assert max_abs(f64(dv2[:L]), f64(dv[sl])) <= 2e-2
        assert max_abs(f64(dk2[:L]), f64(dk[sl])) <= 2e-2
        assert max_abs(f64(dq2[:L]), f64(dq[sl])) <= 2e-2
        s += L
    # without the position-id boundaries (one example over the whole stream) rows differ
    plain = wl.StreamTensors(torch.arange(sum(lens), dtype=torch.int32, device="cuda"),
                             st.q, st.k, st.v, st.dout, [sum(lens)])
    o3, _, _ = run_fwd(plain, w, theta=0.0)
    o4, _, _ = run_fwd(st, w, theta=0.0)
    assert torch.equal(o3[:150], o4[:150])
    assert float((o3[150:] - o4[150:]).abs().max()) > 1e-2
    # and that single-example run is plain causal attention (torch SDPA, fp64, CPU)
    G = Hq // Hkv
    tq, tk, tv = (f64(x) for x in (st.q, st.k, st.v))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(tq).permute(1, 0, 2)[None],
        torch.from_numpy(np.repeat(tk, G, axis=1)).permute(1, 0, 2)[None],
        torch.from_numpy(np.repeat(tv, G, axis=1)).permute(1, 0, 2)[None],
        is_causal=True, scale=w.softmax_scale)[0].permute(1, 0, 2).numpy()
    assert max_abs(f64(o3), ref) <= 1e-2


def test_flat_stream_equals_one_call_per_pack():
    w = wl.workload("c2")
    packs = w.streams[:3]
    flat = [l for p in packs for l in p]
    st = to_cuda(wl.stream_tensors(w, flat, 0))
    out, lse, dq, dk, dv = _run(st, w)
    s = 0
    for p in packs:
        n = sum(p)
        sl = slice(s, s + n)
        one = wl.StreamTensors(st.position_ids[sl].contiguous(), st.q[sl].contiguous(),
                               st.k[sl].contiguous(), st.v[sl].contiguous(),
                               st.dout[sl].contiguous(), p)
        o1, l1, dq1, dk1, dv1 = _run(one, w)
        assert torch.equal(o1, out[sl]) and torch.equal(l1, lse[:, sl])
        assert torch.equal(dk1, dk[sl]) and torch.equal(dv1, dv[sl])
        assert max_abs(f64(dq1), f64(dq[sl])) <= 1e-3
        s += n


def test_reruns_are_bitwise_equal_where_order_is_fixed():
    lens = [700, 33, 129]
    w = wl.Workload("t", 23, 8, 2, 128, 0.0, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0))
    a = _run(st, w)
    b = _run(st, w)
    for i in (0, 1, 3, 4):
        assert torch.equal(a[i], b[i])
    assert max_abs(f64(a[2]), f64(b[2])) <= 1e-3

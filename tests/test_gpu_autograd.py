"""The torch.autograd entry points: same numbers as the library calls they wrap (checked against
the fp64 oracle with the tolerances of the backward tests), and the workspace bookkeeping (plan
and rotated copies reused only when they are the right ones)."""
import numpy as np
import pytest
import torch

from oracle import packed_attention as orc
from oracle import packed_loss as pl
from paper_2407_09105_b200 import autograd as pka, workloads as wl
from helpers import f64, to_cuda

pytestmark = pytest.mark.gpu

TOL_O, TOL_G = 1e-2, 2e-2


def _leafs(st):
    return [t.clone().requires_grad_(True) for t in (st.q, st.k, st.v)]


def _check_layer(st, w, out, grads, theta, window=0):
    pos = st.position_ids.cpu().numpy()
    kw = {"window": window} if window else {}
    o_ref, _ = orc.attn_fwd(f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta, **kw)
    assert (np.abs(f64(out) - o_ref) <= TOL_O + 2.0 ** -8 * np.abs(o_ref)).all()
    refs = orc.attn_bwd(f64(st.dout), f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale, theta,
                        **kw)
    for g, e in zip(grads, refs):
        assert (np.abs(f64(g) - e) <= TOL_G + 2.0 ** -8 * np.abs(e)).all()


@pytest.mark.parametrize("theta", [0.0, 1e4])
def test_two_layers_share_the_workspace(theta, monkeypatch):
    from paper_2407_09105_b200 import api
    seen = []
    real_fwd, real_bwd = api.pk_attn_fwd, api.pk_attn_bwd
    monkeypatch.setattr(api, "pk_attn_fwd", lambda *a, **kw: (seen.append(("f", kw["reuse_plan"])),
                                                              real_fwd(*a, **kw))[1])
    monkeypatch.setattr(api, "pk_attn_bwd", lambda *a, **kw: (seen.append(
        ("b", kw["reuse_plan"], kw["reuse_rotated"])), real_bwd(*a, **kw))[1])
    pka._WORKSPACES.clear()
    lens = [150, 260, 3, 129]
    w = wl.Workload("t", 21, 4, 2, 128, theta, [lens], "test")
    a = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
    b = to_cuda(wl.stream_tensors(w, lens, 1, "cpu"))
    b = wl.StreamTensors(a.position_ids, b.q, b.k, b.v, b.dout, lens)     # same position ids tensor
    la, lb = _leafs(a), _leafs(b)
    ya = pka.packed_attention(*la, a.position_ids, w.softmax_scale, theta)
    yb = pka.packed_attention(*lb, b.position_ids, w.softmax_scale, theta)
    # backward runs layer b first (its rotated copies are still in the workspace), then layer a
    ((ya.float() * a.dout.float()).sum() + (yb.float() * b.dout.float()).sum()).backward()
    _check_layer(a, w, ya.detach(), [t.grad for t in la], theta)
    _check_layer(b, w, yb.detach(), [t.grad for t in lb], theta)
    # one plan for the four calls; only the last layer's backward finds its rotated copies
    assert seen == [("f", False), ("f", True), ("b", True, True), ("b", True, False)]


def test_new_position_ids_are_planned_again():
    w = wl.Workload("t", 22, 2, 2, 64, 1e4, [[1]], "test")
    prev = None
    for lens in ([200, 56], [100, 100, 56], [256]):       # same T, different boundaries
        st = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
        leafs = _leafs(st)
        y = pka.packed_attention(*leafs, st.position_ids, w.softmax_scale, w.rope_theta)
        (y.float() * st.dout.float()).sum().backward()
        _check_layer(st, w, y.detach(), [t.grad for t in leafs], w.rope_theta)
        prev = st
    # ids changed in place (same storage): the version counter forces a new plan
    ids = prev.position_ids
    ids.copy_(torch.tensor(wl.position_ids_from_lengths([128, 128]), dtype=torch.int32))
    st = wl.StreamTensors(ids, prev.q, prev.k, prev.v, prev.dout, [128, 128])
    leafs = _leafs(st)
    y = pka.packed_attention(*leafs, ids, w.softmax_scale, w.rope_theta)
    (y.float() * st.dout.float()).sum().backward()
    _check_layer(st, w, y.detach(), [t.grad for t in leafs], w.rope_theta)


def test_sliding_window_and_default_scale():
    lens = [300, 77]
    w = wl.Workload("t", 23, 4, 1, 128, 0.0, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
    leafs = _leafs(st)
    y = pka.packed_attention(*leafs, st.position_ids.long(), window=100)   # int64 ids are converted
    (y.float() * st.dout.float()).sum().backward()
    assert abs(w.softmax_scale - 128 ** -0.5) < 1e-12
    _check_layer(st, w, y.detach(), [t.grad for t in leafs], 0.0, window=100)
    with pytest.raises(TypeError):
        pka.packed_attention(st.q.float(), st.k, st.v, st.position_ids)


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.float32])
def test_packed_cross_entropy(dtype):
    rng = np.random.default_rng(24)
    lens = (4, 8, 5, 11, 1, 30)
    V = 777
    labels = np.concatenate([np.r_[-100, rng.integers(0, V, size=n - 1)] for n in lens]).astype(np.int64)
    g = torch.Generator(device="cuda").manual_seed(25)
    x = (torch.randn((sum(lens), V), generator=g, device="cuda") * 3).to(dtype).requires_grad_(True)
    loss = pka.packed_cross_entropy(x, torch.tensor(labels, device="cuda"))
    (0.25 * loss).backward()
    x64 = x.detach().float().cpu().numpy().astype(np.float64)
    mean = pl.loss_fwd(x64, labels)[0]
    assert abs(loss.item() - mean) <= 2e-5 * mean + 2e-4
    g_ref = pl.loss_bwd(x64, labels, 0.25)
    tol = (2.0 ** -8 if dtype == torch.bfloat16 else 4e-6) * np.abs(g_ref) + 1e-7
    assert (np.abs(x.grad.float().cpu().numpy() - g_ref) <= tol).all()


def test_attention_into_loss_chain_runs_end_to_end():
    # a one-layer toy: attention -> projection to a vocabulary -> packed loss; the gradient that
    # reaches q equals the attention backward fed with the upstream gradient torch computed
    lens = [90, 40, 126]
    w = wl.Workload("t", 26, 2, 2, 64, 1e4, [lens], "test")
    st = to_cuda(wl.stream_tensors(w, lens, 0, "cpu"))
    T, V = sum(lens), 512
    g = torch.Generator(device="cuda").manual_seed(27)
    W = (torch.randn((2 * 64, V), generator=g, device="cuda") * 0.05).to(torch.bfloat16)
    rng = np.random.default_rng(28)
    labels = torch.tensor(np.concatenate([np.r_[-100, rng.integers(0, V, size=n - 1)] for n in lens]),
                          dtype=torch.int32, device="cuda")
    leafs = _leafs(st)
    y = pka.packed_attention(*leafs, st.position_ids, w.softmax_scale, w.rope_theta)
    y.retain_grad()
    loss = pka.packed_cross_entropy(y.view(T, -1) @ W, labels)
    loss.backward()
    assert torch.isfinite(loss) and all(torch.isfinite(t.grad.float()).all() for t in leafs)
    pos = st.position_ids.cpu().numpy()
    refs = orc.attn_bwd(f64(y.grad), f64(st.q), f64(st.k), f64(st.v), pos, w.softmax_scale,
                        w.rope_theta)
    for got, e in zip([t.grad for t in leafs], refs):
        assert (np.abs(f64(got) - e) <= 2e-2 * np.abs(e).max() + 2.0 ** -8 * np.abs(e)).all()

"""The calls only enqueue work on the given stream (no allocation, no synchronisation, no host
read-back), so a forward + backward can be captured into a CUDA graph and replayed: the replay on
new input values is bitwise what the direct calls give."""
import pytest
import torch

from paper_2407_09105_b200 import api, workloads as wl

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("theta,D", [(0.0, 64), (1e4, 128), (1e4, 96)])
def test_forward_and_backward_replay_from_a_cuda_graph(theta, D):
    lens = [112, 87, 73, 46, 50, 20, 24, 17, 35, 48]
    w = wl.Workload("t", 60, 4, 2, D, theta, [lens], "test")
    st = wl.stream_tensors(w, lens, 0, device="cuda")
    T, Hq, _ = st.q.shape
    ws = api.alloc_workspace(T, Hq, 2, D)
    out = torch.empty_like(st.q)
    lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(st.q), torch.empty_like(st.k), torch.empty_like(st.v)

    def step():
        api.pk_attn_fwd(st.q, st.k, st.v, st.position_ids, w.softmax_scale, theta, out, lse, ws)
        api.pk_attn_bwd(st.dout, st.q, st.k, st.v, out, lse, st.position_ids, w.softmax_scale,
                        theta, dq, dk, dv, ws, reuse_plan=True, reuse_rotated=True)

    step()                                   # warm-up outside the capture (module load, attributes)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    # new values AND new boundaries in the same buffers: the graph replans on the device
    other = wl.stream_tensors(w, [300, 212], 1, device="cuda")
    for dst, src in ((st.q, other.q), (st.k, other.k), (st.v, other.v), (st.dout, other.dout),
                     (st.position_ids, other.position_ids)):
        dst.copy_(src)
    for t in (out, dq, dk, dv):
        t.fill_(float("nan"))
    graph.replay()
    torch.cuda.synchronize()
    got = [t.clone() for t in (out, lse, dq, dk, dv)]
    assert api.pk_status_read(ws) == (api.PK_OK, 0)
    step()
    torch.cuda.synchronize()
    for a, b in zip(got, (out, lse, dq, dk, dv)):
        assert not torch.isnan(a.float()).any()
        assert torch.equal(a, b)

"""CPU checks: the C-ABI library builds, loads and exports every symbol the header
declares; host-side argument validation; the replica helpers under gloo with 2 ranks."""
import ctypes
import os
import re
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "pk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(pk_[a-z_0-9]+)\s*\(", text)))


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2407_09105_b200 import api, build
    path = build.build()
    handle = ctypes.CDLL(path)
    names = _declared_symbols()
    assert {"pk_seqlens_from_posids", "pk_rope_apply", "pk_attn_fwd", "pk_attn_bwd"} <= set(names)
    for n in names:
        assert hasattr(handle, n), n
    assert set(api.EXPORTED_SYMBOLS) == set(names)
    api.lib()


def test_host_only_calls():
    from paper_2407_09105_b200 import api
    assert api.pk_tile_shape() == (128, 128)
    assert api.pk_workspace_bytes(512, 4, 4, 64) > 0
    assert api.pk_workspace_bytes(512, 4, 4, 72) == 0          # head_dim not a multiple of 16
    assert api.pk_workspace_bytes(512, 4, 4, 256) == 0
    # other head sizes run padded: the padded size's workspace plus room for the copies
    assert api.pk_workspace_bytes(512, 4, 4, 80) > api.pk_workspace_bytes(512, 4, 4, 128)
    assert api.pk_workspace_bytes(512, 6, 4, 64) == 0          # Hq % Hkv != 0
    assert api.pk_workspace_bytes(-1, 4, 4, 64) == 0
    offs = [api.pk_workspace_section(s, 1000, 8, 2, 128) for s in range(8)]
    assert all(o % 256 == 0 for o, _ in offs)
    total = api.pk_workspace_bytes(1000, 8, 2, 128)
    assert all(o + n <= total for o, n in offs)
    with pytest.raises(api.PkError):
        api.pk_workspace_section(99, 1000, 8, 2, 128)


def test_argument_validation_returns_codes_without_a_gpu():
    from paper_2407_09105_b200 import api
    L = api.lib()
    # null workspace / negative T / unsupported shapes are rejected before any CUDA call
    assert L.pk_seqlens_from_posids(None, -1, None, None, None, None, 0, None) == api.PK_ERR_INVALID_ARG
    assert L.pk_attn_fwd(None, None, None, None, 16, 4, 4, 72, 1.0, 0.0, 0, None, 0, None, 0, None, 0,
                         None) == api.PK_ERR_UNSUPPORTED
    assert L.pk_attn_fwd(None, None, None, None, 16, 4, 4, 64, -1.0, 0.0, 0, None, 0, None, 0, None, 0,
                         None) == api.PK_ERR_INVALID_ARG
    assert L.pk_attn_fwd(None, None, None, None, 16, 4, 4, 64, 1.0, 0.0, 0, None, 7, None, 0, None, 0,
                         None) == api.PK_ERR_UNSUPPORTED
    assert L.pk_attn_fwd(None, None, None, None, 16, 4, 4, 64, 1.0, 0.0, -1, None, 0, None, 0, None, 0,
                         None) == api.PK_ERR_INVALID_ARG       # negative window
    assert L.pk_attn_bwd(None, None, None, None, None, 0, None, None, 16, 4, 3, 64, 1.0, 0.0, 0, None,
                         None, None, 0, 0, None, 0, None) == api.PK_ERR_UNSUPPORTED
    assert L.pk_rope_apply(None, None, 4, 2, 7, 1e4, 0, None) == api.PK_ERR_UNSUPPORTED
    assert L.pk_seqlens_from_posids_noalloc(1, api.PK_NOALLOC_MAX_TOKENS + 1, 1, None, None,
                                            None) == api.PK_ERR_TOO_LARGE
    assert L.pk_set_timing_events(99, None, None) == api.PK_ERR_INVALID_ARG
    # packed-stream loss: sizes, strides, dtypes and missing outputs
    bad = api.PK_ERR_INVALID_ARG
    assert L.pk_packed_loss_fwd(None, 0, None, -1, 8, 8, -100, None, None, 1, 1, None) == bad
    assert L.pk_packed_loss_fwd(None, 0, None, 4, 0, 0, -100, None, None, 1, 1, None) == bad
    assert L.pk_packed_loss_fwd(None, 0, None, 4, 8, 7, -100, None, None, 1, 1, None) == bad     # stride < V
    assert L.pk_packed_loss_fwd(None, 5, None, 4, 8, 8, -100, None, None, 1, 1, None) == bad     # dtype
    assert L.pk_packed_loss_fwd(None, 0, None, 4, 8, 8, -100, None, None, None, 1, None) == bad  # no result
    assert L.pk_packed_loss_fwd(None, 0, None, 4, 8, 8, -100, None, None, 1, 1, None) == bad     # no logits
    assert L.pk_packed_loss_bwd(None, 0, None, None, None, 1.0, 4, 8, 8, -100, None, None) == bad
    assert L.pk_packed_loss_bwd(None, 0, None, None, 1, 1.0, 0, 8, 8, -100, None, None) == api.PK_OK  # T = 0
    # padded <-> packed
    assert L.pk_pack_rows(None, None, 2, 4, 6, 0, None, None) == bad          # row_bytes
    assert L.pk_pack_rows(None, None, 2, 4, 6, 8, None, None) == bad          # null buffers
    assert L.pk_pack_rows(None, None, 2, 4, 0, 8, None, None) == api.PK_OK    # nothing to move
    assert L.pk_unpack_rows(None, None, -1, 4, 0, 8, None, None) == bad
    assert L.pk_unpack_rows(None, None, 0, 4, 0, 8, None, None) == api.PK_OK


def test_assign_streams_balances_by_pairs():
    from paper_2407_09105_b200 import replicas, workloads as wl
    w = wl.workload("c4")
    pairs = [sum(l * (l + 1) // 2 for l in s) for s in w.streams]
    parts = replicas.assign_streams(pairs, 4)
    assert sorted(i for p in parts for i in p) == list(range(len(pairs)))
    loads = [sum(pairs[i] for i in p) for p in parts]
    assert max(loads) <= 1.25 * (sum(pairs) / 4)
    assert replicas.whole_job_rate(10.0, 4, 2.0) == 20.0


_WORKER = r"""
import os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
from paper_2407_09105_b200 import replicas
dist.init_process_group("gloo")
r = dist.get_rank()
t = replicas.max_over_ranks(10.0 + 5.0 * r, dist)
assert t == 15.0, t
assert replicas.whole_job_rate(3.0, dist.get_world_size(), t) == 6.0 / 15.0
dist.barrier()
dist.destroy_process_group()
print("rank", r, "ok")
"""


def test_replica_timing_max_over_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
           "--master-addr", "127.0.0.1", "--master-port", "29613", str(script), ROOT]
    res = subprocess.run(cmd, capture_output=True, text=True, timeout=240)
    assert res.returncode == 0, res.stdout + res.stderr
    assert res.stdout.count("ok") == 2


def test_reference_arm_other_ranks_do_no_work():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference"],
                         capture_output=True, text=True, timeout=120, env=env)
    assert res.returncode == 0 and res.stdout.strip() == ""

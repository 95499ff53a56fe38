#!/usr/bin/env python
"""Benchmark of the packed-attention hot path on B200.

One step = one pass of the whole path over one packed stream: plan (position_ids ->
cu_seqlens + work lists), forward, delta pre-pass, backward, dQ finishing pass.
Default workload: c4, the Mistral-7B-shaped GQA layer (32 q / 8 kv heads, head_dim 128)
over 16 first-fit-decreasing bins of 8192 tokens, run as one flat stream (bin edges are
example edges, so the result is identical to 16 separate calls).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--impl reference]

Prints ONE JSON line.  `value` is useful TFLOP/s: 14 * D * Hq * sum_e L_e (L_e + 1) / 2
floating-point operations per step (forward 4, backward 10 per causal pair and head
dimension) divided by the device time of the step.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2407_09105_b200 import workloads as wl  # noqa: E402

METRIC = "packed_attn_fwd_bwd_useful_tflops"
UNIT = "TFLOP/s"

# DRAM bytes per causal (query, key, q-head) pair of the dominant (dK/dV) kernel, from the ncu
# capture summarised in profiles/ (scaled to a launch by the number of pairs); None = not captured.
# DRAM bytes per (causal pair, q head) of one launch on the full c4 workload
# (profiles/attn_kernels_c4_full_dram_bytes.txt); other workloads are scaled by their pair count
NCU_BWD_DRAM_BYTES_PER_PAIR = 0.3838   # attn_bwd_dkv_kernel
NCU_DQ_DRAM_BYTES_PER_PAIR = 0.3408    # attn_bwd_dq_kernel
NCU_FWD_DRAM_BYTES_PER_PAIR = 0.2432   # attn_fwd_ws_kernel


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"burst": float(p["bf16_tflops"]), "sustained": float(p["bf16_tflops_sustained"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"burst": 1590.0, "sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for s in self.samples:
            parts = [x.strip() for x in s.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None,
                "sm_max_mhz": float(max(mx)) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def _launches_per_call(theta, Hq, Hkv, D):
    """Kernels of this library per forward+backward pair (default RoPE mode)."""
    if theta <= 0:
        return 5                      # plan, forward, delta, dK/dV, dQ
    # rotated fp16 copies of q and k, made once by the forward:
    return 4 + 4                      # plan, rotate q, rotate k, forward | table, delta, dK/dV, dQ


def _oracle_sample(w: wl.Workload):
    """A bounded sample of whole examples of the workload for the CPU oracle: the example
    closest to 2048 tokens plus the eight shortest ones, all heads."""
    lens = w.flat_lengths()
    order = sorted(range(len(lens)), key=lambda i: lens[i])
    mid = min(range(len(lens)), key=lambda i: abs(lens[i] - 2048))
    pick = sorted(set(order[:8] + [mid]))
    return [lens[i] for i in pick]


def _time_oracle(w: wl.Workload, steps: int = 1):
    """Runs the fp64 numpy oracle (forward + backward) on the sample; returns
    (useful TFLOP/s, seconds per pass, threads, description)."""
    from oracle import packed_attention as orc
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        threads = len(os.sched_getaffinity(0))
    lens = _oracle_sample(w)
    sw = wl.Workload(w.name + "_sample", w.seed, w.num_q_heads, w.num_kv_heads, w.head_dim,
                     w.rope_theta, [lens], w.packing, w.window)
    st = wl.stream_tensors(sw, lens, 0, "cpu")
    q, k, v, do = (x.to(torch.float64).numpy() for x in (st.q, st.k, st.v, st.dout))
    pos = st.position_ids.numpy()
    best = None
    for _ in range(steps):
        t0 = time.perf_counter()
        orc.attn_fwd(q, k, v, pos, sw.softmax_scale, sw.rope_theta, window=w.window)
        orc.attn_bwd(do, q, k, v, pos, sw.softmax_scale, sw.rope_theta, window=w.window)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    flops = sw.useful_flops_fwd + sw.useful_flops_bwd
    desc = (f"{len(lens)} whole examples of {w.name} (lengths {lens}), all {w.num_q_heads} q heads, "
            f"fwd+bwd in fp64 numpy; {sum(lens)} tokens, {flops / 1e9:.1f} useful GFLOP")
    return flops / best / 1e12, best, threads, desc, sum(lens)


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    for _ in range(max(1, min(args.warmup, 1))):
        _time_oracle(w)
    tf = None
    for _ in range(max(1, min(args.steps, 3))):
        tf, dt, threads, desc, toks = _time_oracle(w)
        times.append(dt)
    dt = float(np.mean(times))
    sw_flops = tf * min(times) * 1e12
    value = sw_flops / dt / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": len(times), "warmup": 1, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{w.name} ({w.packing}), bounded sample per step", "Hq": w.num_q_heads,
                   "Hkv": w.num_kv_heads, "head_dim": w.head_dim},
        "tokens_per_s": toks / dt,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                         "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def run_loss(args):
    """`--workload loss`: the packed-stream loss (the step after the model), forward + backward
    over bf16 logits of the first two 8192-token packs of c4 against a 32000-entry vocabulary
    (Mistral / Llama-2 size).  HBM-bound: the forward reads every logit once, the backward
    reads it again and writes its gradient.  Prints one JSON line of its own."""
    from paper_2407_09105_b200 import api
    from oracle import packed_loss as pl
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    w = wl.workload("c4")
    lens = [x for stream in w.streams[:2] for x in stream]
    T, V = sum(lens), 32000
    rng = np.random.default_rng(1234)
    labels_np = np.concatenate([np.r_[-100, rng.integers(0, V, size=n - 1)] for n in lens]).astype(np.int32)
    gen = torch.Generator(device="cuda").manual_seed(99)
    logits = torch.empty((T, V), dtype=torch.bfloat16, device="cuda")
    for i in range(0, T, 2048):                      # bounded temporaries
        n = min(2048, T - i)
        logits[i:i + n] = (torch.randn((n, V), generator=gen, device="cuda") * 2.5).to(torch.bfloat16)
    labels = torch.tensor(labels_np, device="cuda")
    dlogits = torch.empty_like(logits)
    token_loss = torch.empty((T,), device="cuda")
    lse = torch.empty((T,), device="cuda")
    result = torch.empty((2,), device="cuda")
    n_valid = torch.empty((1,), dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def step():
        api.pk_packed_loss_fwd(logits, labels, token_loss, lse, result, n_valid, stream=stream)
        api.pk_packed_loss_bwd(logits, labels, lse, n_valid, 1.0, dlogits, stream=stream)

    kev = {k: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)] for k in (api.PK_KERNEL_LOSS_FWD, api.PK_KERNEL_LOSS_BWD)}
    for pairs in kev.values():                       # torch creates the events on first record
        for a, b in pairs:
            a.record(stream)
            b.record(stream)
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(args.steps):
        for k in kev:
            api.pk_set_timing_events(k, kev[k][i][0], kev[k][i][1])
        step()
    e1.record()
    torch.cuda.synchronize()
    for k in kev:
        api.pk_set_timing_events(k, None, None)
    clocks = sampler.stop()
    ms = e0.elapsed_time(e1) / args.steps
    fwd_ms = float(np.mean([a.elapsed_time(b) for a, b in kev[api.PK_KERNEL_LOSS_FWD]]))
    bwd_ms = float(np.mean([a.elapsed_time(b) for a, b in kev[api.PK_KERNEL_LOSS_BWD]]))
    peaks = _peaks()
    fwd_bytes, bwd_bytes = 2.0 * T * V, 4.0 * T * V
    # end to end: logits from pinned host memory every step, the scalar loss and the gradient back
    e2e = None
    if not args.no_e2e:
        h_logits = torch.empty((T, V), dtype=torch.bfloat16).pin_memory()
        h_logits.copy_(logits)
        h_dl = torch.empty((T, V), dtype=torch.bfloat16).pin_memory()
        h_res = torch.empty((2,)).pin_memory()
        n_e2e = max(2, min(args.steps, 5))
        torch.cuda.synchronize()
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(n_e2e):
            logits.copy_(h_logits, non_blocking=True)
            step()
            h_dl.copy_(dlogits, non_blocking=True)
            h_res.copy_(result, non_blocking=True)
        a1.record()
        torch.cuda.synchronize()
        e_ms = a0.elapsed_time(a1) / n_e2e
        e2e = {"value": T / (e_ms * 1e-3), "unit": "tokens/s", "ms_per_step": e_ms,
               "h2d_bytes_per_step": int(fwd_bytes), "d2h_bytes_per_step": int(fwd_bytes) + 8}
    cpu = None
    if not args.no_cpu_baseline:
        rows = 256                                    # whole leading examples would be too slow
        x = logits[:rows].float().cpu().numpy().astype(np.float64)
        t0 = time.perf_counter()
        pl.loss_fwd(x, labels_np[:rows])
        pl.loss_bwd(x, labels_np[:rows])
        dt = time.perf_counter() - t0
        cpu = {"value": rows / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
               "sample": f"first {rows} rows of the stream, forward + backward in fp64 numpy"}
    line = {
        "metric": "packed_loss_fwd_bwd_tokens_per_s", "value": T / (ms * 1e-3), "unit": "tokens/s",
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic",
        "config": {"workload": "loss: first 2 packs of c4 (16363 tokens) x vocabulary 32000, bf16 logits",
                   "tokens": T, "vocab": V, "l2": "inputs_exceed_l2"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": 3 * args.steps,
        "roofline": {"kernel": "ce_bwd_kernel", "bound": "hbm", "achieved": bwd_bytes / (bwd_ms * 1e-3) / 1e9,
                     "peak": peaks["hbm_gbs"], "peak_kind": "copy bandwidth, " + peaks["source"],
                     "unit": "GB/s", "frac": bwd_bytes / (bwd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                     # 3.9039 B per logit: profiles/loss_kernels_2packs_vocab32000.txt (read + write)
                     "traffic": 3.9039 * T * V, "ms_per_launch": bwd_ms,
                     "fwd_kernel": {"achieved": fwd_bytes / (fwd_ms * 1e-3) / 1e9,
                                    "frac": fwd_bytes / (fwd_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                                    "ms_per_launch": fwd_ms}},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))


def run_pack(args):
    """`--workload pack`: padded batch <-> packed stream for hidden-state rows (4096 bf16 = 8 KB per
    token) of the first 8 mini-batches of c3 (16 examples each, padded to the longest of the
    mini-batch), one call per mini-batch and direction.  HBM-bound copies; one JSON line."""
    from paper_2407_09105_b200 import api
    from oracle import pad_pack as pp
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    w = wl.workload("c3")
    batches = w.streams[:8]
    H = 4096
    gen = torch.Generator(device="cuda").manual_seed(5)
    items = []
    for lens in batches:
        B, lmax, T = len(lens), max(lens), sum(lens)
        cu = torch.tensor(np.concatenate([[0], np.cumsum(lens)]), dtype=torch.int32, device="cuda")
        padded = torch.randn((B, lmax, H), generator=gen, device="cuda").to(torch.bfloat16)
        items.append((cu, padded, torch.empty((T, H), dtype=torch.bfloat16, device="cuda"),
                      torch.empty_like(padded)))
    T_all = sum(sum(l) for l in batches)
    rows_padded = sum(len(l) * max(l) for l in batches)
    rb = H * 2
    stream = torch.cuda.current_stream()

    def step_pack():
        for cu, padded, packed, back in items:
            api.pk_pack_rows(padded, cu, packed, stream=stream)

    def step_unpack():
        for cu, padded, packed, back in items:
            api.pk_unpack_rows(packed, cu, back, stream=stream)

    def timed(fn):
        for _ in range(max(args.warmup, 3)):
            fn()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record()
        for _ in range(args.steps):
            fn()
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b) / args.steps

    ms_pack, ms_unpack = timed(step_pack), timed(step_unpack)
    peaks = _peaks()
    pack_bytes = 2.0 * T_all * rb
    unpack_bytes = (T_all + rows_padded) * float(rb)
    cpu = None
    if not args.no_cpu_baseline:
        cu, padded, packed, back = items[0]
        x = padded.float().cpu().numpy()
        t0 = time.perf_counter()
        y = pp.pack_rows(x, batches[0])
        pp.unpack_rows(y, batches[0], max(batches[0]))
        dt = time.perf_counter() - t0
        cpu = {"value": sum(batches[0]) / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
               "sample": "first mini-batch, pack + unpack in numpy"}
    ms = ms_pack + ms_unpack
    line = {
        "metric": "pad_pack_roundtrip_tokens_per_s", "value": T_all / (ms * 1e-3), "unit": "tokens/s",
        "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8",
        "data": "synthetic",
        "config": {"workload": "pack: 8 mini-batches of c3 (16 examples each), 8 KB rows, pack then unpack",
                   "tokens": T_all, "padded_rows": rows_padded, "row_bytes": rb, "l2": "inputs_exceed_l2"},
        "e2e": None, "gpu_launches": 2 * len(items) * args.steps,
        "roofline": {"kernel": "rows_move_kernel<16, unpack>", "bound": "hbm",
                     "achieved": unpack_bytes / (ms_unpack * 1e-3) / 1e9, "peak": peaks["hbm_gbs"],
                     "peak_kind": "copy bandwidth, " + peaks["source"], "unit": "GB/s",
                     "frac": unpack_bytes / (ms_unpack * 1e-3) / 1e9 / peaks["hbm_gbs"], "traffic": None,
                     "ms_per_step": ms_unpack,
                     "pack": {"achieved": pack_bytes / (ms_pack * 1e-3) / 1e9,
                              "frac": pack_bytes / (ms_pack * 1e-3) / 1e9 / peaks["hbm_gbs"],
                              "ms_per_step": ms_pack}},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--packs", type=int, default=0,
                    help="use only the first N packs of the workload (small cases for profiling)")
    ap.add_argument("--per-stream", action="store_true",
                    help="one call per pack / mini-batch instead of one flat stream")
    ap.add_argument("--window", type=int, default=0,
                    help="sliding-window attention: keys visible per row (0 = all, the default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl != "reference" else args.warmup

    if args.workload == "loss":
        run_loss(args)
        return
    if args.workload == "pack":
        run_pack(args)
        return
    w = wl.workload(args.workload)
    if args.packs > 0:
        w = wl.Workload(f"{w.name}[:{args.packs}]", w.seed, w.num_q_heads, w.num_kv_heads,
                        w.head_dim, w.rope_theta, w.streams[:args.packs], w.packing)
    if args.window > 0:
        w = wl.Workload(f"{w.name}+window{args.window}", w.seed, w.num_q_heads, w.num_kv_heads,
                        w.head_dim, w.rope_theta, w.streams, w.packing, args.window)
    if args.impl == "reference":
        run_reference(args, w)
        return

    from paper_2407_09105_b200 import api, replicas

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # every rank works on its own replica of the workload (different values, same lengths)
    lens = w.flat_lengths()
    st = wl.stream_tensors(w, lens, stream_index=rank, device="cuda")
    T, Hq, D = st.q.shape
    Hkv = st.k.shape[1]
    scale, theta = w.softmax_scale, w.rope_theta
    out = torch.empty_like(st.q)
    lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
    dq, dk, dv = torch.empty_like(st.q), torch.empty_like(st.k), torch.empty_like(st.v)
    stream = torch.cuda.current_stream()

    if args.per_stream:
        # one call per packed stream (mini-batch / pack), all on the same CUDA stream: the same
        # tokens as the flat run, cut at the stream edges
        bounds = np.concatenate([[0], np.cumsum([sum(x) for x in w.streams])]).tolist()
        ws = api.alloc_workspace(max(b - a for a, b in zip(bounds, bounds[1:])), Hq, Hkv, D)
        pieces = []
        for a, b in zip(bounds, bounds[1:]):
            n = b - a
            pieces.append((st.q[a:b], st.k[a:b], st.v[a:b], st.dout[a:b], st.position_ids[a:b],
                           out[a:b], torch.empty((Hq, n), dtype=torch.float32, device="cuda"),
                           dq[a:b], dk[a:b], dv[a:b]))

        def step():
            for (q_, k_, v_, do_, pos_, out_, lse_, dq_, dk_, dv_) in pieces:
                api.pk_attn_fwd(q_, k_, v_, pos_, scale, theta, out_, lse_, ws,
                                reuse_plan=False, window=w.window, stream=stream)
                api.pk_attn_bwd(do_, q_, k_, v_, out_, lse_, pos_, scale, theta,
                                dq_, dk_, dv_, ws, reuse_plan=True, reuse_rotated=True, window=w.window, stream=stream)
        calls_per_step = len(pieces)
    else:
        ws = api.alloc_workspace(T, Hq, Hkv, D)

        def step():
            api.pk_attn_fwd(st.q, st.k, st.v, st.position_ids, scale, theta, out, lse, ws,
                            reuse_plan=False, window=w.window, stream=stream)
            api.pk_attn_bwd(st.dout, st.q, st.k, st.v, out, lse, st.position_ids, scale, theta,
                            dq, dk, dv, ws, reuse_plan=True, reuse_rotated=True, window=w.window, stream=stream)
        calls_per_step = 1

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    code, detail = api.pk_status_read(ws)
    if code != api.PK_OK:
        raise SystemExit(f"device status {code} (detail {detail})")

    # per-kernel events: recorded by the library around the two main kernels
    kev = {k: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
               for _ in range(args.steps)]
           for k in (api.PK_KERNEL_FWD, api.PK_KERNEL_BWD, api.PK_KERNEL_BWD_DQ)}
    for pairs in kev.values():
        for a, b in pairs:
            a.record(stream)
            b.record(stream)
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(args.steps):
        if calls_per_step == 1:
            for k, pairs in kev.items():
                api.pk_set_timing_events(k, pairs[i][0], pairs[i][1])
        step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    for k in kev:
        api.pk_set_timing_events(k, None, None)
    ms_step = replicas.max_over_ranks(e0.elapsed_time(e1), dist, "cuda") / args.steps
    fwd_ms = float(np.mean([a.elapsed_time(b) for a, b in kev[api.PK_KERNEL_FWD]]))
    bwd_ms = float(np.mean([a.elapsed_time(b) for a, b in kev[api.PK_KERNEL_BWD]]))
    # two backward kernels (dK/dV, dQ): bench.py never selects the in-tile RoPE mode, whose single
    # backward kernel would be timed as PK_KERNEL_BWD alone
    split = True
    dq_ms = float(np.mean([a.elapsed_time(b) for a, b in kev[api.PK_KERNEL_BWD_DQ]])) if split else 0.0

    flops_step = w.useful_flops_fwd + w.useful_flops_bwd
    value = world * flops_step / (ms_step * 1e-3) / 1e12
    tokens_per_s = world * T / (ms_step * 1e-3)

    # ---- end to end: host buffers in, host buffers out, through the same calls ------------
    e2e = None
    if not args.no_e2e:
        host_in = [x.cpu().pin_memory() for x in (st.q, st.k, st.v, st.dout, st.position_ids)]
        dev_in = [st.q, st.k, st.v, st.dout, st.position_ids]
        dev_out = [out, dq, dk, dv]
        host_out = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in dev_out]
        h2d = sum(x.numel() * x.element_size() for x in host_in)
        d2h = sum(x.numel() * x.element_size() for x in host_out)

        # One pack at a time through paper_2407_09105_b200.pipeline: copy-in of pack i+1, kernels of
        # pack i and copy-out of pack i-1 overlap (three streams); a single flat stream has
        # nothing to overlap with and goes copy -> kernels -> copy.
        from paper_2407_09105_b200 import pipeline
        bounds = np.concatenate([[0], np.cumsum([sum(x) for x in w.streams])]).tolist()
        spans = list(zip(bounds, bounds[1:]))
        if len(spans) > 1:
            cut = lambda ts: [[x[a:b] for x in ts] for a, b in spans]
            ws_p = api.alloc_workspace(max(b - a for a, b in spans), Hq, Hkv, D)
            lse_p = [torch.empty((Hq, b - a), dtype=torch.float32, device="cuda") for a, b in spans]

            def compute(i, s):
                a, b = spans[i]
                api.pk_attn_fwd(st.q[a:b], st.k[a:b], st.v[a:b], st.position_ids[a:b], scale, theta,
                                out[a:b], lse_p[i], ws_p, reuse_plan=False, window=w.window, stream=s)
                api.pk_attn_bwd(st.dout[a:b], st.q[a:b], st.k[a:b], st.v[a:b], out[a:b], lse_p[i],
                                st.position_ids[a:b], scale, theta, dq[a:b], dk[a:b], dv[a:b], ws_p,
                                reuse_plan=True, reuse_rotated=True, window=w.window, stream=s)

            pipe = pipeline.HostPipeline(cut(host_in), cut(dev_in), cut(dev_out), cut(host_out), compute)

            def e2e_step():
                pipe.step(stream)
        else:
            def e2e_step():
                for h, d in zip(host_in, dev_in):
                    d.copy_(h, non_blocking=True)
                step()
                for d, h in zip(dev_out, host_out):
                    h.copy_(d, non_blocking=True)

        n_e2e = max(3, min(args.steps, 5))
        e2e_step()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        ms_e2e = replicas.max_over_ranks(a.elapsed_time(b), dist, "cuda") / n_e2e
        e2e = {"value": world * flops_step / (ms_e2e * 1e-3) / 1e12, "unit": UNIT,
               "ms_per_step": ms_e2e, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
               "how": ("one pack at a time, copies overlapped with kernels on three streams"
                       if len(spans) > 1 else "copy in, kernels, copy out on one stream")}

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peaks = _peaks()
    if calls_per_step > 1:      # per-kernel events are recorded for the flat run only
        fwd_ms = bwd_ms = dq_ms = float('nan')
    # The backward (10*D FLOPs per causal pair and q head: S, dP, dV, dK, dQ) dominates the step.
    # Without in-tile RoPE it runs as two launches, dK/dV (S, dP, dV, dK: 8*D) and dQ (S and dP once
    # more, and dQ: 6*D executed, 2*D of them new), so the roofline entry takes the two together:
    # the paper's 10*D per pair over the sum of their durations.  The per-launch figures follow.
    bwd_both_ms = bwd_ms + dq_ms
    bwd_tflops = w.useful_flops_bwd / (bwd_both_ms * 1e-3) / 1e12
    per_pair = Hq * w.causal_pairs
    fwd_tflops = w.useful_flops_fwd / (fwd_ms * 1e-3) / 1e12
    traffic = None
    if split and NCU_BWD_DRAM_BYTES_PER_PAIR is not None and NCU_DQ_DRAM_BYTES_PER_PAIR is not None:
        traffic = (NCU_BWD_DRAM_BYTES_PER_PAIR + NCU_DQ_DRAM_BYTES_PER_PAIR) * per_pair
    roofline = {
        "kernel": ("attn_bwd_dkv_kernel + attn_bwd_dq_kernel (the backward)" if split
                   else "attn_bwd_kernel"),
        "bound": "tensor", "achieved": bwd_tflops,
        "peak": peaks["sustained"], "peak_kind": f"bf16 sustained, {peaks['source']}",
        "peak_burst": peaks["burst"], "unit": "TFLOP/s", "frac": bwd_tflops / peaks["sustained"],
        "traffic": traffic, "ms_per_launch": bwd_both_ms, "launches_per_step": 2 if split else 1,
        "note": ("algorithmic FLOPs = 10*D per causal pair and q head over both launches; each "
                 "launch's own figures below count what it executes" if split else "in-tile RoPE kernel"),
        "bwd_dkv_kernel": ({"executed_tflops": 8 * D * per_pair / (bwd_ms * 1e-3) / 1e12,
                            "frac_executed": 8 * D * per_pair / (bwd_ms * 1e-3) / 1e12 / peaks["sustained"],
                            "ms_per_launch": bwd_ms,
                            "traffic": (None if NCU_BWD_DRAM_BYTES_PER_PAIR is None
                                        else NCU_BWD_DRAM_BYTES_PER_PAIR * per_pair)}
                           if split else None),
        "bwd_dq_kernel": ({"executed_tflops": 6 * D * per_pair / (dq_ms * 1e-3) / 1e12,
                           "frac_executed": 6 * D * per_pair / (dq_ms * 1e-3) / 1e12 / peaks["sustained"],
                           "ms_per_launch": dq_ms,
                           "traffic": (None if NCU_DQ_DRAM_BYTES_PER_PAIR is None
                                       else NCU_DQ_DRAM_BYTES_PER_PAIR * per_pair)}
                          if split else None),
        "fwd_kernel": {"achieved": fwd_tflops, "frac": fwd_tflops / peaks["sustained"],
                       "ms_per_launch": fwd_ms,
                       "traffic": NCU_FWD_DRAM_BYTES_PER_PAIR * per_pair if split else None},
    }
    cpu_baseline = None
    if not args.no_cpu_baseline:
        tf, dt, threads, desc, _ = _time_oracle(w)
        cpu_baseline = {"value": tf, "unit": UNIT, "cores": threads, "kind": "oracle",
                        "sample": desc, "seconds": dt}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": (f"{w.name}: {w.packing}, {len(w.streams)} packs, " +
                                ("one call per pack" if args.per_stream else "as one flat stream")),
                   "tokens": T, "examples": len(lens), "Hq": Hq, "Hkv": Hkv, "head_dim": D,
                   "rope_theta": theta, "window": w.window, "causal_pairs": w.causal_pairs,
                   "flop_convention": "14*D*Hq*sum L(L+1)/2", "l2": "inputs_exceed_l2",
                   "replicas": world},
        "tokens_per_s": tokens_per_s,
        "pct_of_bf16_peak": {"sustained": 100 * value / world / peaks["sustained"],
                             "burst": 100 * value / world / peaks["burst"],
                             "source": peaks["source"]},
        "clocks": clocks, "e2e": e2e, "gpu_launches": _launches_per_call(theta, Hq, Hkv, D) * args.steps * calls_per_step,
        "roofline": roofline if calls_per_step == 1 else None, "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""torch.autograd entry points over the library calls: what a training loop calls instead of a
padded attention and a padded loss (Sec. 3.4: the flattened mini-batch goes through the model with
its position ids, nothing else changes).

Plumbing only -- buffers, the workspace and the bookkeeping of what it holds; every computation is
a library call of ``api``.  One workspace per device is kept and grown on demand; all layers of a
model share it, so its plan is reused whenever the position ids are the same tensor, unchanged,
and the rotated copies of q and k are reused by the backward of the call that made them when no
other call came in between (the last layer, typically).  The calls of a device must therefore be
ordered on the GPU (one CUDA stream, or events between streams), as a training loop's are.
"""
from __future__ import annotations

import math
from typing import Dict, Optional, Tuple

import torch

from . import api


class _Workspace:
    """The workspace of one device and what its sections currently hold."""

    def __init__(self) -> None:
        self.buf: Optional[torch.Tensor] = None
        self.shape: Tuple[int, int, int, int] = (0, 0, 0, 0)
        self.plan_key: Optional[tuple] = None      # position ids the plan was made from
        self.plan_ids: Optional[torch.Tensor] = None   # ... kept alive, so their address stays theirs
        self.rotated_owner: int = -1               # forward call whose rotated copies are there
        self.calls: int = 0

    def fit(self, T: int, Hq: int, Hkv: int, D: int, device) -> torch.Tensor:
        # the section layout depends on the shape, so a plan does not survive a change of shape
        if self.buf is None or self.shape != (T, Hq, Hkv, D) or self.buf.device != device:
            need = api.pk_workspace_bytes(T, Hq, Hkv, D)
            if need == 0:
                raise api.PkError("pk_workspace_bytes", api.PK_ERR_UNSUPPORTED)
            if self.buf is None or self.buf.numel() < need or self.buf.device != device:
                self.buf = torch.empty(need, dtype=torch.uint8, device=device)
            self.shape = (T, Hq, Hkv, D)
            self.plan_key = self.plan_ids = None
            self.rotated_owner = -1
        return self.buf

    def planned(self, position_ids: torch.Tensor) -> bool:
        """True when the plan in the workspace was made from these position ids.  Remembers them
        for the next call either way."""
        key = (position_ids.data_ptr(), position_ids.numel(), position_ids._version)
        same = self.plan_key == key
        self.plan_key, self.plan_ids = key, position_ids
        return same


_WORKSPACES: Dict[int, _Workspace] = {}


def _workspace(device: torch.device) -> _Workspace:
    idx = device.index if device.index is not None else torch.cuda.current_device()
    return _WORKSPACES.setdefault(idx, _Workspace())


class _PackedAttention(torch.autograd.Function):
    @staticmethod
    def forward(ctx, q, k, v, position_ids, softmax_scale, rope_theta, window):
        q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
        T, Hq, D = q.shape
        Hkv = k.shape[1]
        st = _workspace(q.device)
        ws = st.fit(T, Hq, Hkv, D, q.device)
        out = torch.empty_like(q)
        lse = torch.empty((Hq, T), dtype=torch.float32, device=q.device)
        api.pk_attn_fwd(q, k, v, position_ids, softmax_scale, rope_theta, out, lse, ws,
                        reuse_plan=st.planned(position_ids), window=window)
        st.calls += 1
        st.rotated_owner = st.calls
        ctx.call = st.calls
        ctx.args = (softmax_scale, rope_theta, window)
        ctx.save_for_backward(q, k, v, out, lse, position_ids)
        return out

    @staticmethod
    def backward(ctx, dout):
        q, k, v, out, lse, position_ids = ctx.saved_tensors
        softmax_scale, rope_theta, window = ctx.args
        T, Hq, D = q.shape
        st = _workspace(q.device)
        ws = st.fit(T, Hq, k.shape[1], D, q.device)
        planned = st.planned(position_ids)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        api.pk_attn_bwd(dout.contiguous(), q, k, v, out, lse, position_ids, softmax_scale,
                        rope_theta, dq, dk, dv, ws, reuse_plan=planned,
                        reuse_rotated=(planned and st.rotated_owner == ctx.call), window=window)
        st.rotated_owner = -1          # the backward uses that section for its own copies
        return dq, dk, dv, None, None, None, None


def packed_attention(q: torch.Tensor, k: torch.Tensor, v: torch.Tensor,
                     position_ids: torch.Tensor, softmax_scale: Optional[float] = None,
                     rope_theta: float = 0.0, window: int = 0) -> torch.Tensor:
    """Causal attention of a packed stream, every example on its own (boundaries from
    ``position_ids``, the paragraph after Table 1): ``q`` [T, Hq, D], ``k``/``v`` [T, Hkv, D] bf16
    on the GPU, ``position_ids`` int32 [T].  ``rope_theta`` > 0 rotates q and k by position id
    inside the call (gradients are for the un-rotated tensors); ``window`` > 0 limits every row to
    its ``window`` most recent keys.  Differentiable in q, k, v."""
    for name, t in (("q", q), ("k", k), ("v", v)):
        if t.dtype != torch.bfloat16 or not t.is_cuda or t.dim() != 3:
            raise TypeError(f"{name} must be a bf16 CUDA tensor [T, H, D]")
    if softmax_scale is None:
        softmax_scale = 1.0 / math.sqrt(q.shape[-1])
    if position_ids.dtype != torch.int32:
        position_ids = position_ids.to(torch.int32)
    return _PackedAttention.apply(q, k, v, position_ids.contiguous().view(-1), float(softmax_scale),
                                  float(rope_theta), int(window))


class _PackedLoss(torch.autograd.Function):
    @staticmethod
    def forward(ctx, logits, labels, ignore_index):
        T = logits.shape[0]
        dev = logits.device
        token_loss = torch.empty((T,), dtype=torch.float32, device=dev)
        lse = torch.empty((T,), dtype=torch.float32, device=dev)
        result = torch.empty((2,), dtype=torch.float32, device=dev)
        n_valid = torch.empty((1,), dtype=torch.int32, device=dev)
        api.pk_packed_loss_fwd(logits, labels, token_loss, lse, result, n_valid,
                               ignore_index=ignore_index)
        ctx.ignore_index = ignore_index
        ctx.save_for_backward(logits, labels, lse, n_valid)
        return result[0].clone()

    @staticmethod
    def backward(ctx, grad):
        logits, labels, lse, n_valid = ctx.saved_tensors
        dlogits = torch.empty_strided(logits.shape, logits.stride(), dtype=logits.dtype,
                                      device=logits.device)
        # the library takes the upstream gradient by value: one host read of a scalar per step
        api.pk_packed_loss_bwd(logits, labels, lse, n_valid, float(grad), dlogits,
                               ignore_index=ctx.ignore_index)
        return dlogits, None, None


def packed_cross_entropy(logits: torch.Tensor, labels: torch.Tensor,
                         ignore_index: int = -100) -> torch.Tensor:
    """Mean next-token loss of a packed stream (Sec. 3.5): row t is scored against
    ``labels[t + 1]``; the collator's ``ignore_index`` at every example start keeps an example's
    last row from predicting the next example's first token.  ``logits`` [T, V] bf16 or fp32 with
    unit stride in V, ``labels`` int32 [T].  Differentiable in ``logits``."""
    if labels.dtype != torch.int32:
        labels = labels.to(torch.int32)
    return _PackedLoss.apply(logits, labels.contiguous().view(-1), int(ignore_index))

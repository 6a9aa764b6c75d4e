"""Data-parallel form of the training step: sequences sharded over ranks, the LM head replicated.

Every stage of the path is per token except the masked mean of Eq. 2, so a job that splits its
sequences over ranks only has to agree on M = sum_r M_r (the number of valid tokens in the whole
job) and add up the LM-head gradient:

    M_r                 = a3po_mask_count(mask_r)                     before the step (the mask is an input)
    M                   = all_reduce(M_r, SUM)                        one int64
    scale_r             = M_r / M                                     a3po_dp_loss_scale
    L_r, grad_r         = a3po_train_step(..., loss_scale=scale_r)    gradients come out weighted by M_r / M
    grad_w              = all_reduce(grad_w_r, SUM)                   the only large exchange (V x H fp32)
    L                   = all_reduce(scale_r * L_r, SUM)

grad_hidden and grad_logp stay on their rank (they belong to that rank's tokens).  The collectives
are torch.distributed's (NCCL on GPUs); no kernel of the library reads another GPU's memory.

`DataParallelStep` is written against three callables so that the same reduction logic runs on
GPUs (the library's calls) and, in the CPU tests, on the fp64 oracle under the gloo backend.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


class DataParallelStep:
    """count_fn(mask) -> int64 tensor [1];  scale_fn(m_local, m_global, loss_local or None) -> (scale [1], weighted
    loss [1] or None);  step_fn(batch, scale) -> dict with at least "loss" [1] and "grad_w" (accumulated or fresh)."""

    def __init__(self, count_fn, scale_fn, step_fn, group=None):
        self.count_fn, self.scale_fn, self.step_fn, self.group = count_fn, scale_fn, step_fn, group

    def _world(self):
        return dist.get_world_size(self.group) if dist.is_available() and dist.is_initialized() else 1

    def __call__(self, batch):
        m_local = self.count_fn(batch["mask"])
        m_global = m_local.clone()
        if self._world() > 1:
            dist.all_reduce(m_global, op=dist.ReduceOp.SUM, group=self.group)
        scale, _ = self.scale_fn(m_local, m_global, None)
        out = self.step_fn(batch, scale)
        _, weighted = self.scale_fn(m_local, m_global, out["loss"])
        if self._world() > 1:
            dist.all_reduce(out["grad_w"], op=dist.ReduceOp.SUM, group=self.group)
            dist.all_reduce(weighted, op=dist.ReduceOp.SUM, group=self.group)
        out["loss_local"] = out["loss"]
        out["loss"] = weighted
        out["m_local"], out["m_global"], out["scale"] = m_local, m_global, scale
        return out


def gpu_data_parallel_step(group=None):
    """The step on this rank's GPU through the library.  `batch` holds the device tensors of a3po_train_step
    (hidden, w, targets, behav_logp, versions, current_version, adv, mask, clip_eps) and its output / scratch
    tensors (logp, lse, grad_logp, loss, grad_hidden, grad_w, ws, optionally stats, entropy, status)."""
    from . import binding as b

    def count_fn(mask):
        count = torch.zeros(1, dtype=torch.int64, device=mask.device)
        ws = b.new_workspace(b.a3po_mask_count_workspace_bytes(), mask.device)
        b.a3po_mask_count(mask, count, ws)
        return count

    def scale_fn(m_local, m_global, loss_local):
        scale = torch.empty(1, dtype=torch.float32, device=m_local.device)
        weighted = torch.empty(1, dtype=torch.float32, device=m_local.device) if loss_local is not None else None
        b.a3po_dp_loss_scale(m_local, m_global, scale, loss_local=loss_local, weighted_loss=weighted)
        return scale, weighted

    def step_fn(x, scale):
        b.a3po_train_step(x["hidden"], x["w"], x["targets"], x["behav_logp"], x["versions"], x["current_version"],
                          x["adv"], x["mask"], x["clip_eps"], x["logp"], x["lse"], x["grad_logp"], x["loss"],
                          x["grad_hidden"], x["grad_w"], x["ws"], stats=x.get("stats"), entropy=x.get("entropy"),
                          loss_scale=scale, accumulate_grad_w=x.get("accumulate_grad_w", False),
                          status=x.get("status"))
        return {"loss": x["loss"], "grad_w": x["grad_w"], "grad_hidden": x["grad_hidden"], "grad_logp": x["grad_logp"]}

    return DataParallelStep(count_fn, scale_fn, step_fn, group)

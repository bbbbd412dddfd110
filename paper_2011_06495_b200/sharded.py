"""Worker-sharded majority-vote step: the N workers are spread over the ranks of a process group.

Every arithmetic step runs in the CUDA library (mv_vote, mv_select, mv_aggregate_partial,
mv_finish_mean); this module only strings them together with the two exchanges the method has when
workers live on different GPUs: the vote counts are summed over the ranks (the parameter server's
count of Eq. 9) and so are the partial sums on the shared mask (the all-reduce the paper points out
under Eq. 8).  With one rank it degenerates to the single-GPU step.
"""
from __future__ import annotations

import contextlib
from typing import Optional

import torch
import torch.distributed as dist


class ShardedStep:
    """ctx: an MvContext-like object sized for (N_total, d, K); group: a torch.distributed process group
    (None = the default group); N_total: workers over all ranks.

    The library enqueues on the stream the context was created with, the collectives on torch's current
    stream: `step` makes the context's stream current for its whole body, so the two are one stream and
    every call sees the results of the one before it."""

    def __init__(self, ctx, N_total: int, d: int, K: int, device, group: Optional[dist.ProcessGroup] = None):
        self.ctx, self.N_total, self.d, self.K, self.group = ctx, int(N_total), int(d), int(K), group
        self.votes = torch.empty(d, dtype=torch.uint8, device=device)
        self.partial = torch.empty(K, dtype=torch.float64, device=device)

    def step(self, grads_local: torch.Tensor, err_local: torch.Tensor, out_idx: torch.Tensor, out_val: torch.Tensor):
        """grads_local, err_local: this rank's [N_local, d] rows; err_local is updated in place to the
        residual; out_idx / out_val [K] receive the shared mask and the mean over all N_total workers."""
        if self.N_total > 255:
            raise ValueError("at most 255 workers in total (votes are counted in a byte)")
        with self._on_context_stream():
            self.ctx.mv_vote(grads_local, err_local, votes=self.votes, K=self.K)
            dist.all_reduce(self.votes, op=dist.ReduceOp.SUM, group=self.group)
            self.ctx.mv_select(self.votes, self.N_total, out_idx, K=self.K)
            self.ctx.mv_aggregate_partial(err_local, out_idx, self.partial)
            dist.all_reduce(self.partial, op=dist.ReduceOp.SUM, group=self.group)
            self.ctx.mv_finish_mean(self.partial, self.N_total, out_val)

    def _on_context_stream(self):
        stream = getattr(self.ctx, "stream", None)
        if isinstance(stream, torch.cuda.Stream):
            return torch.cuda.stream(stream)
        return contextlib.nullcontext()      # a CPU stand-in for the context has no stream

"""Data-parallel form of the stage step (Section 3.1, last paragraph; Section 4.1): every worker
runs mslt_step_backward on its share of the batch, the gradients of the trainable slice only are
summed over the workers, every worker applies the same update.  One process per GPU,
torch.distributed (NCCL) for the exchange; the frozen bottom layers exchange nothing.

Only argument marshalling and the collective calls live here: the step itself, the normalisation
by the global slot count and the optimizer run in the library's kernels.
"""
from __future__ import annotations


def reduce_buckets(buckets, dist, group=None):
    """Sums every tensor of `buckets` over the workers, in place."""
    for b in buckets:
        dist.all_reduce(b, op=dist.ReduceOp.SUM, group=group)


class DataParallelStep:
    """Drives one model replica of a data-parallel job.

    step(): (1) the number of valid MLM slots is summed over the workers, so that every worker
    divides its loss terms and gradients by the global count; (2) mslt_step_backward, with a hook that
    starts the all-reduce of a gradient bucket on a second stream as soon as the backward pass has
    finished that bucket: the output layer's gradients travel while the top layers are still in
    their backward pass, and so on down; (3) mslt_step_apply, which waits for the reductions;
    (4) the workers' loss shares are summed.  With one worker the collectives are skipped.
    """

    def __init__(self, model, dist=None, group=None, overlap: bool = True):
        import torch
        self.torch, self.m, self.group = torch, model, group
        self.dist = dist if dist is not None and dist.is_available() and dist.is_initialized() else None
        self.world = self.dist.get_world_size(group) if self.dist else 1
        self.comm = torch.cuda.Stream(device=model.device) if (self.world > 1 and overlap) else None
        self.buckets = None
        self.reduced = 0          # buckets handed to the collective in the last step
        self.bytes_exchanged = 0  # gradient bytes this worker contributed in the last step
        if self.comm is not None:  # stays set: mslt_step_apply waits for the communication stream
            model.mslt_set_bucket_hook(self.comm, self._hook)

    def _hook(self, i: int):
        with self.torch.cuda.stream(self.comm):
            self.dist.all_reduce(self.buckets[i], op=self.dist.ReduceOp.SUM, group=self.group)
        self.reduced += 1

    def step(self, tokens, seq_lens, mlm_positions, mlm_labels, read_loss: bool = True):
        torch, m = self.torch, self.m
        with torch.cuda.stream(m.stream):
            total = ((mlm_positions >= 0) & (mlm_labels >= 0)).sum().to(torch.int32).reshape(1)
            if self.world > 1:
                self.dist.all_reduce(total, op=self.dist.ReduceOp.SUM, group=self.group)
            self.buckets = m.grad_buckets()
            self.reduced = 0
            self.bytes_exchanged = 4 * sum(b.numel() for b in self.buckets) if self.world > 1 else 0
            m.mslt_step_backward(tokens, seq_lens, mlm_positions, mlm_labels, total_valid=total, sync=False)
            if self.world > 1 and self.comm is None:
                reduce_buckets(self.buckets, self.dist, self.group)
            m.mslt_step_apply()
            if not read_loss:      # nothing is synchronised: the caller reads the loss later, if at all
                return None
            loss = torch.tensor([m.mslt_read_loss()], device=m.device)
            if self.world > 1:
                self.dist.all_reduce(loss, op=self.dist.ReduceOp.SUM, group=self.group)
        return float(loss.item())

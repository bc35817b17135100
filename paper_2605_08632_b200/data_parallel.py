"""Row-sharded data parallelism for the CAT loss.

Draft blocks are independent (the product of Eq. 10 never crosses a block), so a batch shards
by whole blocks across ranks with the head weight W replicated.  What has to be exchanged is
what the batch mean of Eq. 11 and the weight gradient sum over rows: the number of valid rows
N (before the backward pass, so every rank scales its gradients by g / N_global), dW (summed),
and the weighted loss sums.  dH stays local.

One process per GPU; `torch.distributed` (NCCL on GPUs) does the exchange.  With
`overlap=True` the two-call path is used and the all-reduce of each vocabulary slab of dW is
enqueued on a side stream as soon as the library reports that slab final
(cat_loss_bwd_events), so the transfer runs under the GEMMs of the following slabs.  The three
scalar operations that combine per-rank counts and losses are plain tensor arithmetic on
one-element tensors; every step of the loss itself runs in the library's kernels.

The arithmetic of the loss lives in an *engine* object (count_valid / forward_backward /
forward + backward_slabs).  `CudaEngine` is the product's; tests on machines without a GPU
plug in an engine of their own to exercise the exchange logic over gloo.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import binding as B
from .api import CatLoss

__all__ = ["CudaEngine", "DataParallelCatLoss", "shard_rows"]


def shard_rows(T: int, K: int, world: int, rank: int) -> tuple[int, int]:
    """Rows [begin, end) of rank `rank`: whole draft blocks, as even as possible."""
    if T % K:
        raise ValueError("T must be a multiple of K")
    blocks = T // K
    base, extra = divmod(blocks, world)
    b0 = rank * base + min(rank, extra)
    b1 = b0 + base + (1 if rank < extra else 0)
    return b0 * K, b1 * K


class CudaEngine:
    """The local loss on this rank's rows, through the C library."""

    def __init__(self, T_local: int, d: int, V: int, K: int, dtype=torch.bfloat16, dW_dtype=torch.float32, slab_mib: int = 0):
        self.cl = CatLoss(T_local, d, V, K, dtype=dtype, dW_dtype=dW_dtype, slab_mib=slab_mib)
        self.device = self.cl.loss.device
        self._n = torch.zeros(1, dtype=torch.int64, device=self.device)
        self.slabs = B.cat_loss_bwd_slabs(self.cl.shape)
        self._events = [torch.cuda.Event() for _ in range(len(self.slabs) - 1)]

    def count_valid(self, labels, valid):
        B.cat_count_valid(self.cl.shape, labels, valid, self._n)
        return self._n

    def forward_backward(self, H, W, labels, valid, grad_loss, conf_ext=None):
        loss, dH, dW = self.cl.forward_backward(H, W, labels, valid, conf_ext=conf_ext, grad_loss=grad_loss)
        return loss, dH, dW

    def forward(self, H, W, labels, valid, conf_ext=None):
        return self.cl.forward(H, W, labels, valid, conf_ext)

    def backward_slabs(self, H, W, labels, valid, grad_loss):
        """Backward pass; returns (dH, dW, [(v0, v1, event)]): rows v0:v1 of dW are final once `event` has fired."""
        cl = self.cl
        B.cat_loss_bwd_events(cl.shape, H, W, labels, valid, cl.lse, cl.weight, grad_loss, cl.dH, cl.dW, False, cl.ws_bwd,
                              self._events)
        return cl.dH, cl.dW, [(self.slabs[i], self.slabs[i + 1], self._events[i]) for i in range(len(self._events))]


class DataParallelCatLoss:
    """Global CAT loss and gradients over rows sharded across the ranks of `group`."""

    def __init__(self, engine, group=None, overlap: bool = False):
        self.engine = engine
        self.group = group
        self.overlap = overlap and hasattr(engine, "backward_slabs")
        self._comm_stream = None

    def step(self, H, W, labels, valid=None, g: float = 1.0, conf_ext=None):
        """Returns (loss, dH_local, dW): loss and dW are the global ones (identical on all ranks),
        dH belongs to this rank's rows; all scaled by g / N_global."""
        eng = self.engine
        n_local = eng.count_valid(labels, valid)                       # int64 [1]
        n_global = n_local.clone()
        dist.all_reduce(n_global, op=dist.ReduceOp.SUM, group=self.group)
        # the library scales local gradients by grad_loss / N_local; make that g / N_global
        grad_loss = (float(g) * n_local.to(torch.float32) / n_global.clamp(min=1).to(torch.float32)).contiguous()
        if self.overlap:
            loss_local = eng.forward(H, W, labels, valid, conf_ext)
            dH, dW, parts = eng.backward_slabs(H, W, labels, valid, grad_loss)
            if self._comm_stream is None:
                self._comm_stream = torch.cuda.Stream(device=dW.device)
            main = torch.cuda.current_stream(dW.device)
            with torch.cuda.stream(self._comm_stream):
                for v0, v1, ev in parts:
                    self._comm_stream.wait_event(ev)
                    dist.all_reduce(dW[v0:v1], op=dist.ReduceOp.SUM, group=self.group)
            main.wait_stream(self._comm_stream)
        else:
            loss_local, dH, dW = eng.forward_backward(H, W, labels, valid, grad_loss, conf_ext=conf_ext)
            dist.all_reduce(dW, op=dist.ReduceOp.SUM, group=self.group)
        # loss_local = S_local / N_local  ->  global mean = sum_ranks S_local / N_global
        part = loss_local.to(torch.float64) * n_local.to(torch.float64) / n_global.clamp(min=1).to(torch.float64)
        dist.all_reduce(part, op=dist.ReduceOp.SUM, group=self.group)
        return part.to(torch.float32), dH, dW

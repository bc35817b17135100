"""Convenience layer over the binding: owns the device buffers of one problem shape.

It allocates outputs and workspaces with torch once, then every call goes straight to the
C entry points.  No arithmetic of the method happens here.
"""
from __future__ import annotations

import torch

from . import binding as B


class CatLoss:
    """Buffers and calls for one (T, d, V, K, dtype) problem on the current CUDA device."""

    def __init__(self, T: int, d: int, V: int, K: int, dtype: torch.dtype = torch.bfloat16,
                 dW_dtype: torch.dtype = torch.float32, slab_mib: int = 0, device: str = "cuda",
                 fixed_decay_gamma: float | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("CatLoss needs a CUDA device; there is no CPU path")
        code = {torch.bfloat16: B.CAT_BF16, torch.float32: B.CAT_F32}
        self.dtype, self.dW_dtype = dtype, dW_dtype
        if fixed_decay_gamma is None:
            self.shape = B.make_shape(T, d, V, K, code[dtype], code[dW_dtype], slab_mib=slab_mib)
        else:   # the fixed position decay the paper compares CAT with: weight gamma^k
            self.shape = B.make_shape(T, d, V, K, code[dtype], code[dW_dtype], slab_mib=slab_mib,
                                      weight_mode=B.CAT_WEIGHT_FIXED_DECAY, decay_gamma=float(fixed_decay_gamma))
        self.T, self.d, self.V, self.K = T, d, V, K
        dev = torch.device(device)
        nf, nb = B.cat_loss_workspace_bytes(self.shape, 0), B.cat_loss_workspace_bytes(self.shape, 1)
        if nf == 0 or nb == 0:
            raise ValueError("invalid shape for cat_loss")
        self.ws_fwd = torch.empty(nf, dtype=torch.uint8, device=dev)
        self.ws_bwd = torch.empty(nb, dtype=torch.uint8, device=dev)
        self._ws_fused = None
        self._ws_kd = None
        self.loss3 = None
        self.loss = torch.zeros(1, dtype=torch.float32, device=dev)
        self.lse = torch.empty(T, dtype=torch.float32, device=dev)
        self.conf = torch.empty(T, dtype=torch.float32, device=dev)
        self.weight = torch.empty(T, dtype=torch.float32, device=dev)
        self.stats = torch.zeros(32, dtype=torch.uint8, device=dev)
        self.dH = torch.empty(T, d, dtype=dtype, device=dev)
        self.dW = torch.empty(V, d, dtype=dW_dtype, device=dev)

    def forward(self, H, W, labels, valid=None, conf_ext=None):
        B.cat_loss_fwd(self.shape, H, W, labels, valid, conf_ext, self.loss, self.lse, self.conf, self.weight,
                       self.stats, self.ws_fwd)
        return self.loss

    def backward(self, H, W, labels, valid=None, grad_loss=None, accumulate_dW=False):
        B.cat_loss_bwd(self.shape, H, W, labels, valid, self.lse, self.weight, grad_loss, self.dH, self.dW,
                       accumulate_dW, self.ws_bwd)
        return self.dH, self.dW

    def forward_backward(self, H, W, labels, valid=None, conf_ext=None, grad_loss=None, accumulate_dW=False):
        """cat_loss_fwd_bwd: one call, logits kept per row slab instead of recomputed."""
        if self._ws_fused is None:
            n = B.cat_loss_workspace_bytes(self.shape, 2)
            self._ws_fused = torch.empty(n, dtype=torch.uint8, device=self.loss.device)
        B.cat_loss_fwd_bwd(self.shape, H, W, labels, valid, conf_ext, grad_loss, self.loss, self.lse, self.conf,
                           self.weight, self.stats, self.dH, self.dW, accumulate_dW, self._ws_fused)
        return self.loss, self.dH, self.dW

    def forward_backward_timed(self, H, W, labels, valid=None, conf_ext=None, grad_loss=None, accumulate_dW=False):
        """cat_loss_fwd_bwd_events: same results as forward_backward; returns the stage events
        (start, set-up, then per row slab: label reference, logits GEMM, row kernel, slab preparation,
        dH GEMM, dW GEMM; finalize)."""
        if self._ws_fused is None:
            n = B.cat_loss_workspace_bytes(self.shape, 2)
            self._ws_fused = torch.empty(n, dtype=torch.uint8, device=self.loss.device)
        n_slabs = len(B.cat_loss_fused_slabs(self.shape)) - 1
        events = [torch.cuda.Event(enable_timing=True) for _ in range(6 * n_slabs + 3)]
        B.cat_loss_fwd_bwd_events(self.shape, H, W, labels, valid, conf_ext, grad_loss, self.loss, self.lse, self.conf,
                                  self.weight, self.stats, self.dH, self.dW, accumulate_dW, self._ws_fused, events)
        return events

    def accept_len(self) -> torch.Tensor:
        """cat_accept_len: per-block estimate of the expected acceptance length (Eq. 8) from the
        conf / weight of the last forward."""
        out = torch.empty(self.T // self.K, dtype=torch.float32, device=self.loss.device)
        B.cat_accept_len(self.shape, self.conf, self.weight, out)
        return out

    def kd_forward_backward(self, H, W, labels, valid, Ht, Wt, block_start_host, beta, conf_source=B.CAT_CONF_TARGET,
                            conf_ext=None, grad_loss=None, accumulate_dW=False):
        """cat_kd_loss_fwd_bwd: Eq. 12, CAT-weighted cross-entropy + distillation from the target head.
        Returns (loss3, dH, dW) with loss3 = [total, cross-entropy part, distillation part]."""
        desc = B.make_kd_desc(Ht.shape[0], Ht.shape[1], float(beta), conf_source, ldHt=Ht.stride(0), ldWt=Wt.stride(0))
        n = B.cat_kd_workspace_bytes(self.shape, desc, block_start_host)
        if n == 0:
            raise ValueError("invalid problem for cat_kd_loss_fwd_bwd")
        if self._ws_kd is None or self._ws_kd.numel() < n:
            self._ws_kd = torch.empty(n, dtype=torch.uint8, device=self.loss.device)
        if self.loss3 is None:
            self.loss3 = torch.zeros(3, dtype=torch.float32, device=self.loss.device)
        B.cat_kd_loss_fwd_bwd(self.shape, desc, H, W, labels, valid, Ht, Wt, block_start_host, conf_ext, grad_loss,
                              self.loss3, self.lse, self.conf, self.weight, self.stats, self.dH, self.dW, accumulate_dW,
                              self._ws_kd)
        return self.loss3, self.dH, self.dW

    def kd_status(self) -> int:
        return int(self._ws_kd[:4].view(torch.int32).item())

    def fused_status(self) -> int:
        return int(self._ws_fused[:4].view(torch.int32).item())

    def bwd_status(self) -> int:
        return int(self.ws_bwd[:4].view(torch.int32).item())

    def fwd_stats(self):
        return B.read_stats(self.stats)


class TargetConfidence:
    """Buffers and calls for cat_conf_fwd / cat_conf_window: target-model confidences of L
    sequence positions (Eq. 9) and their layout as draft rows (Eq. 12)."""

    def __init__(self, L: int, d: int, V: int, dtype: torch.dtype = torch.bfloat16, device: str = "cuda"):
        if not torch.cuda.is_available():
            raise RuntimeError("TargetConfidence needs a CUDA device; there is no CPU path")
        code = {torch.bfloat16: B.CAT_BF16, torch.float32: B.CAT_F32}
        self.L = L
        self.shape = B.make_shape(L, d, V, 1, code[dtype])
        n = B.cat_loss_workspace_bytes(self.shape, 3)
        if n == 0:
            raise ValueError("invalid shape for cat_conf_fwd")
        dev = torch.device(device)
        self.ws = torch.empty(n, dtype=torch.uint8, device=dev)
        self.conf_seq = torch.empty(L, dtype=torch.float32, device=dev)
        self.lse_seq = torch.empty(L, dtype=torch.float32, device=dev)

    def forward(self, Ht, Wt, labels, valid=None):
        B.cat_conf_fwd(self.shape, Ht, Wt, labels, valid, self.conf_seq, self.lse_seq, self.ws)
        return self.conf_seq

    def window(self, block_start: torch.Tensor, K: int) -> torch.Tensor:
        n_blocks = block_start.numel()
        out = torch.empty(n_blocks * K, dtype=torch.float32, device=self.conf_seq.device)
        B.cat_conf_window(self.conf_seq, self.L, block_start, n_blocks, K, out)
        return out

    def status(self) -> int:
        return int(self.ws[:4].view(torch.int32).item())


class _CatLossFn(torch.autograd.Function):
    """autograd glue: the loss and both gradients come out of one cat_loss_fwd_bwd call in forward();
    backward() hands them over, multiplied by the incoming scalar gradient when that is not 1.
    The gradient buffers the call wrote become the graph node's own and the engine gets fresh ones,
    so a second call through the same engine before backward() cannot overwrite them."""

    @staticmethod
    def forward(ctx, H, W, labels, valid, conf_ext, K, engine):
        loss, dH, dW = engine.forward_backward(H.detach(), W.detach(), labels, valid, conf_ext=conf_ext)
        engine.dH, engine.dW = torch.empty_like(dH), torch.empty_like(dW)
        ctx.save_for_backward(dH, dW)
        return loss.clone().reshape(())

    @staticmethod
    def backward(ctx, grad_out):
        dH, dW = ctx.saved_tensors
        if bool((grad_out == 1).item()):
            return dH, dW, None, None, None, None, None
        return dH * grad_out.to(dH.dtype), dW * grad_out.to(dW.dtype), None, None, None, None, None


class CatLossModule(torch.nn.Module):
    """Drop-in loss head for a draft-model training loop: `loss = head(H, labels, valid)` with
    H [T, d] the hidden states of the draft positions (T = blocks * K), using `weight` [V, d] as the
    LM head.  The library's dW is float32; autograd casts it to the parameter's dtype when it stores
    it in `weight.grad`.  An upstream gradient other than 1 is applied by a tensor multiply in
    backward() (chain-rule glue; pass `grad_loss` to CatLoss.forward_backward to have the kernels
    apply a scale instead).  One engine (buffers for one T) is kept per distinct T."""

    def __init__(self, weight: torch.Tensor, K: int, slab_mib: int = 0):
        super().__init__()
        self.weight = weight if isinstance(weight, torch.nn.Parameter) else torch.nn.Parameter(weight)
        self.K = K
        self.slab_mib = slab_mib
        self._engines = {}

    def forward(self, H, labels, valid=None, conf_ext=None):
        T, d = H.shape
        eng = self._engines.get(T)
        if eng is None:
            eng = self._engines[T] = CatLoss(T, d, self.weight.shape[0], self.K, dtype=H.dtype, slab_mib=self.slab_mib,
                                             device=str(H.device))
        return _CatLossFn.apply(H, self.weight, labels, valid, conf_ext, self.K, eng)

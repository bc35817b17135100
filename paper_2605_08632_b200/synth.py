"""Seeded synthetic draft-training batches for the CAT loss.

This module only draws inputs (hidden states H, head weight W, labels, the
valid-row mask).  It holds none of the method's arithmetic, so both the CUDA
path and the CPU oracle may be fed from it.  The batches stand in for the
paper's training corpora and draft-model activations, which need datasets and
trained weights; shapes follow public Llama-3.2-1B/3B and Qwen3-0.6B head sizes
and the paper's draft lengths K (Table 5, Table 6).

Draw order per config is fixed: H, W, labels, biased-row choice, valid mask.
Everything is drawn in float32 on the CPU from one torch.Generator and cast to
the config's dtype afterwards.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

__all__ = ["CONFIGS", "Batch", "make_batch", "zipf_labels", "TargetSide", "make_target_side"]


@dataclass(frozen=True)
class ConfigSpec:
    name: str
    T: int
    K: int
    d: int
    V: int
    dtype: str          # "f32" or "bf16"
    seed: int
    labels: str         # "uniform" or "zipf"
    bias: tuple | None  # (fraction of rows, low, high) label-logit bias, or None
    invalid: float      # fraction of rows masked invalid


CONFIGS = {
    1: ConfigSpec("tiny_f32", 512, 8, 256, 4096, "f32", 0, "uniform", None, 0.0),
    2: ConfigSpec("llama1b_head", 16384, 8, 2048, 128256, "bf16", 1, "uniform", None, 0.0),
    3: ConfigSpec("qwen06b_head_k16", 32768, 16, 1024, 151936, "bf16", 2, "zipf", None, 0.0),
    4: ConfigSpec("realistic_conf", 65536, 8, 2048, 128256, "bf16", 3, "uniform", (0.6, 6.0, 6.0), 0.10),
    5: ConfigSpec("large_stream_k32", 131072, 32, 3072, 128256, "bf16", 4, "zipf", None, 0.0),
    # variant of 4 whose bias is spread over [6, 18] so that confidences really reach ~1
    41: ConfigSpec("realistic_conf_wide", 65536, 8, 2048, 128256, "bf16", 3, "uniform", (0.6, 6.0, 18.0), 0.10),
}


@dataclass
class Batch:
    spec: ConfigSpec
    T: int
    K: int
    d: int
    V: int
    H: torch.Tensor        # [T, d] spec dtype
    W: torch.Tensor        # [V, d] spec dtype
    labels: torch.Tensor   # [T] int64
    valid: torch.Tensor    # [T] uint8
    biased: torch.Tensor   # [T] bool, rows whose label logit was raised

    @property
    def torch_dtype(self):
        return torch.float32 if self.spec.dtype == "f32" else torch.bfloat16


def zipf_labels(n: int, V: int, s: float, gen: torch.Generator) -> torch.Tensor:
    """Token ids with Zipf(s) frequencies over a seeded random permutation of the vocabulary."""
    perm = torch.randperm(V, generator=gen)
    ranks = np.arange(1, V + 1, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-s))
    cdf /= cdf[-1]
    u = torch.rand(n, generator=gen, dtype=torch.float64).numpy()
    idx = np.minimum(np.searchsorted(cdf, u, side="left"), V - 1)
    return perm[torch.from_numpy(idx)]


def _valid_mask(T: int, K: int, frac: float, gen: torch.Generator) -> torch.Tensor:
    """About `frac` of rows invalid: half as block-end tails (some whole blocks), half as holes."""
    valid = torch.ones(T, dtype=torch.uint8)
    if frac <= 0.0:
        return valid
    B = T // K
    # block-end tails: tail length U{1..K}, mean (K+1)/2; choose blocks so tails cover frac/2 of rows
    p_block = (frac / 2.0) * K / ((K + 1) / 2.0)
    pick = torch.rand(B, generator=gen) < p_block
    tail = torch.randint(1, K + 1, (B,), generator=gen)
    pos = torch.arange(K).unsqueeze(0).expand(B, K)
    tail_mask = pick.unsqueeze(1) & (pos >= (K - tail).unsqueeze(1))
    holes = torch.rand(T, generator=gen) < (frac / 2.0)
    valid[tail_mask.reshape(-1) | holes] = 0
    return valid


def make_batch(cfg: int, T: int | None = None, d: int | None = None, V: int | None = None,
               K: int | None = None) -> Batch:
    """Draw config `cfg`; T/d/V/K may be overridden to get a reduced case of the same recipe."""
    spec = CONFIGS[cfg]
    T = spec.T if T is None else T
    d = spec.d if d is None else d
    V = spec.V if V is None else V
    K = spec.K if K is None else K
    if T % K:
        raise ValueError("T must be a multiple of K")
    gen = torch.Generator(device="cpu").manual_seed(spec.seed)
    H = torch.randn(T, d, generator=gen, dtype=torch.float32)
    W = torch.randn(V, d, generator=gen, dtype=torch.float32) * 0.02
    if spec.labels == "uniform":
        labels = torch.randint(0, V, (T,), generator=gen, dtype=torch.int64)
    else:
        labels = zipf_labels(T, V, 1.1, gen)
    dt = torch.float32 if spec.dtype == "f32" else torch.bfloat16
    W = W.to(dt)
    biased = torch.zeros(T, dtype=torch.bool)
    if spec.bias is not None:
        frac, lo, hi = spec.bias
        biased = torch.rand(T, generator=gen) < frac
        amount = lo + (hi - lo) * torch.rand(T, generator=gen)
        # raise the label logit of the chosen rows by `amount`: H_r += amount * W[y_r] / |W[y_r]|^2
        rows = torch.nonzero(biased).squeeze(1)
        Wy = W[labels[rows]].double()
        scale = amount[rows].double() / (Wy * Wy).sum(dim=1)
        H[rows] += (Wy * scale.unsqueeze(1)).float()
    H = H.to(dt)
    valid = _valid_mask(T, K, spec.invalid, gen)
    if spec.invalid > 0:
        labels = torch.where(valid.bool(), labels, torch.full_like(labels, -100))
    return Batch(spec, T, K, d, V, H.contiguous(), W.contiguous(), labels.contiguous(), valid, biased)


@dataclass
class TargetSide:
    """Inputs of the target-model side for a batch: one flattened training sequence of L
    positions whose drafted continuations are the batch's blocks."""
    L: int
    d_t: int
    Ht: torch.Tensor            # [L, d_t] target final hidden states
    Wt: torch.Tensor            # [V, d_t] target LM head
    seq_labels: torch.Tensor    # [L] int64: token that follows each position's prefix
    block_start: torch.Tensor   # [T / K] int64: sequence index of each block's first drafted token


def make_target_side(batch: Batch, d_t: int = 0, seed_offset: int = 7919) -> TargetSide:
    """Target-side stand-ins for `batch`: one block per prefix position n = 0..B-1 of a sequence
    of L = B + K - 1 positions, block n drafting positions n..n+K-1 (Eq. 12's (n, k) grid).  The
    labels of the draft rows are NOT changed; seq_labels[n + k] is set to the label of row
    (n, 0) for k = 0 and drawn for the tail, so they are only consistent along k = 0 -- enough
    for a synthetic head, whose rows are independent draws anyway."""
    spec = batch.spec
    d_t = d_t or batch.d
    nb = batch.T // batch.K
    L = nb + batch.K - 1
    gen = torch.Generator(device="cpu").manual_seed(spec.seed + seed_offset)
    Ht = torch.randn(L, d_t, generator=gen, dtype=torch.float32)
    Wt = torch.randn(batch.V, d_t, generator=gen, dtype=torch.float32) * 0.02
    tail = torch.randint(0, batch.V, (batch.K - 1,), generator=gen, dtype=torch.int64)
    first = batch.labels.reshape(nb, batch.K)[:, 0].clamp(min=0)
    seq_labels = torch.cat([first, tail]).contiguous()
    dt = batch.torch_dtype
    Wt = Wt.to(dt)
    # make the target fairly sure of about half of the positions, so window products are not all ~V^-k
    sure = torch.rand(L, generator=gen) < 0.5
    amount = 4.0 + 10.0 * torch.rand(L, generator=gen)
    rows = torch.nonzero(sure).squeeze(1)
    Wy = Wt[seq_labels[rows]].double()
    Ht[rows] += (Wy * (amount[rows].double() / (Wy * Wy).sum(dim=1)).unsqueeze(1)).float()
    return TargetSide(L, d_t, Ht.to(dt).contiguous(), Wt.contiguous(), seq_labels, torch.arange(nb, dtype=torch.int64))

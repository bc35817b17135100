"""Out-of-bounds writes, checked without a sanitizer: every output and the workspace of each
entry point sits between guard zones filled with a sentinel byte, inside one arena; after the
call the guards must be untouched.  Shapes are ragged in every dimension (rows, hidden size,
vocabulary, last slab), which is where a tile-based kernel would overrun."""
import numpy as np
import pytest
import torch

from paper_2605_08632_b200 import binding as B
from paper_2605_08632_b200 import synth

pytestmark = pytest.mark.gpu
GUARD = 4096
SENTINEL = 0xA5


class Arena:
    """One device buffer; carve() hands out 256-byte aligned views separated by guard zones."""

    def __init__(self, nbytes):
        self.buf = torch.full((nbytes,), SENTINEL, dtype=torch.uint8, device="cuda")
        self.off = GUARD
        self.spans = []

    def carve(self, shape, dtype):
        n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
        start = (self.off + 255) // 256 * 256
        assert start + n + GUARD <= self.buf.numel(), "arena too small"
        self.spans.append((start, start + n))
        self.off = start + n + GUARD
        return self.buf[start:start + n].view(dtype).view(*shape)

    def check(self):
        mask = torch.ones(self.buf.numel(), dtype=torch.bool, device="cuda")
        for a, b in self.spans:
            mask[a:b] = False
        bad = (self.buf != SENTINEL) & mask
        assert not bool(bad.any()), f"guard bytes overwritten near offset {int(torch.nonzero(bad)[0])}"


@pytest.mark.parametrize("cfg,kw", [(41, dict(T=1000, d=200, V=5000)), (41, dict(T=24 * 5, d=136, V=1001 - 1, K=5)), (1, dict(T=136, d=36, V=520))])
def test_no_entry_point_writes_outside_its_buffers(cfg, kw):
    batch = synth.make_batch(cfg, **kw)
    T, d, V, K = batch.T, batch.d, batch.V, batch.K
    dt = batch.torch_dtype
    bf16 = dt == torch.bfloat16
    shape = B.make_shape(T, d, V, K, B.CAT_BF16 if bf16 else B.CAT_F32, slab_mib=1)
    ws_sizes = [B.cat_loss_workspace_bytes(shape, p) for p in (0, 1, 2, 3)]
    ts = synth.make_target_side(batch, d_t=72) if bf16 else None
    kd_desc = B.make_kd_desc(ts.L, ts.d_t, 0.1) if bf16 else None
    kd_ws = B.cat_kd_workspace_bytes(shape, kd_desc, ts.block_start) if bf16 else 0
    esz = 2 if bf16 else 4
    total = sum(ws_sizes) + kd_ws + T * d * esz + V * d * 4 + 8 * T * 4 + (1 << 20)
    ar = Arena(total)
    loss = ar.carve((3,), torch.float32)
    lse, conf, weight = (ar.carve((T,), torch.float32) for _ in range(3))
    stats = ar.carve((32,), torch.uint8)
    dH = ar.carve((T, d), dt)
    dW = ar.carve((V, d), torch.float32)
    acc_len = ar.carve((T // K,), torch.float32)
    conf_ext = ar.carve((T,), torch.float32)
    n_valid = ar.carve((1,), torch.int64)
    wss = [ar.carve((n,), torch.uint8) for n in ws_sizes]
    ws_kd = ar.carve((kd_ws,), torch.uint8) if bf16 else None
    dev = "cuda"
    H, W, y, v = batch.H.to(dev), batch.W.to(dev), batch.labels.to(dev), batch.valid.to(dev)

    B.cat_loss_fwd(shape, H, W, y, v, None, loss[:1], lse, conf, weight, stats, wss[0])
    B.cat_loss_bwd(shape, H, W, y, v, lse, weight, None, dH, dW, False, wss[1])
    B.cat_loss_fwd_bwd(shape, H, W, y, v, None, None, loss[:1], lse, conf, weight, stats, dH, dW, True, wss[2])
    B.cat_accept_len(shape, conf, weight, acc_len)
    B.cat_count_valid(shape, y, v, n_valid)
    B.cat_conf_fwd(shape, H, W, y, v, conf, lse, wss[3])
    starts = torch.arange(T // K, dtype=torch.int64, device=dev)
    B.cat_conf_window(conf, T, starts, T // K, K, conf_ext)
    if bf16:
        B.cat_kd_loss_fwd_bwd(shape, kd_desc, H, W, y, v, ts.Ht.to(dev), ts.Wt.to(dev), ts.block_start, None, None, loss, lse,
                              conf, weight, stats, dH, dW, False, ws_kd)
    torch.cuda.synchronize()
    ar.check()
    assert torch.isfinite(dH.float()).all() and torch.isfinite(dW).all() and torch.isfinite(loss).all()

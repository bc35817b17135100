"""Row-sharded data parallelism: the exchange logic over gloo with two CPU processes (an
oracle-backed engine stands in for the CUDA library, which cannot run here), and on a GPU the
product engine with a one-rank NCCL group, including the slab-wise overlapped dW all-reduce."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import cat_oracle as O
from paper_2605_08632_b200 import synth
from paper_2605_08632_b200.data_parallel import DataParallelCatLoss, shard_rows


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


class OracleEngine:
    """Local loss through the fp64 oracle (CPU).  Mirrors the library's convention: local
    gradients are scaled by grad_loss / N_local and the local loss is S_local / N_local."""

    def __init__(self, K):
        self.K = K

    def count_valid(self, labels, valid):
        V = self.V
        return torch.tensor([int(O.effective_valid(labels, valid, V).sum())], dtype=torch.int64)

    def forward_backward(self, H, W, labels, valid, grad_loss, conf_ext=None):
        fwd, dH, dW = O.cat_forward_backward(H, W, labels, valid, self.K, conf_ext=conf_ext, g=float(grad_loss.item()))
        return torch.tensor([fwd["loss"]], dtype=torch.float64), torch.from_numpy(dH), torch.from_numpy(dW)


def _worker(rank, world, port, cfg_kw, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    batch = synth.make_batch(41, **cfg_kw)
    r0, r1 = shard_rows(batch.T, batch.K, world, rank)
    eng = OracleEngine(batch.K)
    eng.V = batch.V
    dp = DataParallelCatLoss(eng)
    loss, dH, dW = dp.step(batch.H[r0:r1].double(), batch.W.double(), batch.labels[r0:r1], batch.valid[r0:r1], g=0.7)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), loss=loss.numpy(), dH=dH.numpy(), dW=dW.numpy(), r0=r0, r1=r1)
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [2, 3])
def test_sharded_ranks_reproduce_the_single_process_result(tmp_path, world):
    cfg_kw = dict(T=8 * 11, d=16, V=64)          # 11 blocks: uneven shards, masked rows (config 41 recipe)
    mp.spawn(_worker, args=(world, _free_port(), cfg_kw, str(tmp_path)), nprocs=world, join=True)
    batch = synth.make_batch(41, **cfg_kw)
    fwd, dH, dW = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, g=0.7)
    covered = 0
    for rank in range(world):
        z = np.load(os.path.join(str(tmp_path), f"rank{rank}.npz"))
        assert abs(float(z["loss"][0]) - fwd["loss"]) <= 1e-6 * abs(fwd["loss"])     # loss returned as float32
        # the per-rank scale g * N_local / N_global travels as a binary32 scalar (the library's grad_loss): 1e-7 relative
        assert np.linalg.norm(z["dW"] - dW) <= 1e-6 * np.linalg.norm(dW)             # summed over ranks
        r0, r1 = int(z["r0"]), int(z["r1"])
        assert np.linalg.norm(z["dH"] - dH[r0:r1]) <= 1e-6 * np.linalg.norm(dH[r0:r1])   # local rows, global scale
        assert r0 % batch.K == 0 and r1 % batch.K == 0
        covered += r1 - r0
    assert covered == batch.T


def test_shard_rows_covers_all_blocks_once():
    for T, K, world in [(80, 8, 3), (16, 16, 4), (4096, 8, 8)]:
        spans = [shard_rows(T, K, world, r) for r in range(world)]
        assert spans[0][0] == 0 and spans[-1][1] == T
        assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        assert max(e - b for b, e in spans) - min(e - b for b, e in spans) <= K


@pytest.mark.gpu
@pytest.mark.parametrize("overlap", [False, True])
def test_cuda_engine_one_rank_nccl_group(overlap):
    from paper_2605_08632_b200.data_parallel import CudaEngine
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(_free_port())
    torch.cuda.set_device(0)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        batch = synth.make_batch(41, T=768, d=256, V=6000)
        eng = CudaEngine(batch.T, batch.d, batch.V, batch.K, slab_mib=2)        # several vocabulary slabs
        if overlap:
            assert len(eng.slabs) - 1 >= 3
        dp = DataParallelCatLoss(eng, overlap=overlap)
        dev = "cuda"
        loss, dH, dW = dp.step(batch.H.to(dev), batch.W.to(dev), batch.labels.to(dev), batch.valid.to(dev), g=0.7)
        torch.cuda.synchronize()
        fwd, dH_o, dW_o = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, g=0.7)
        assert abs(loss.item() - fwd["loss"]) <= 1e-3 * fwd["loss"]
        assert np.linalg.norm(dH.float().cpu().numpy() - dH_o) <= 1e-2 * np.linalg.norm(dH_o)
        assert np.linalg.norm(dW.float().cpu().numpy() - dW_o) <= 1e-2 * np.linalg.norm(dW_o)
        n = torch.zeros(1, dtype=torch.int64, device=dev)
        from paper_2605_08632_b200 import binding as B
        B.cat_count_valid(eng.cl.shape, batch.labels.to(dev), batch.valid.to(dev), n)
        assert int(n.item()) == fwd["n_valid"]
    finally:
        dist.destroy_process_group()

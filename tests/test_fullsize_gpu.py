"""Full-size parity in the launch configuration bench.py times (default slab sizes).

The oracle cannot afford every output at these sizes, so it computes sampled ones exactly:
whole draft blocks (lse, confidence, weight and the dH rows of those blocks) for configs 2-5,
and for config 2, the benchmark workload, the whole forward pass (exact loss, every lse and
weight) plus sampled dW rows.  On top come properties that hold at any size: the weights are
the binary32 product of the GPU's own confidences for every row, dW sums to zero over the
vocabulary, masked rows have zero dH, and the loss equals the fp64 reduction of the per-row
outputs.  Both entry-point paths are checked: cat_loss_fwd + cat_loss_bwd and cat_loss_fwd_bwd.
"""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2605_08632_b200 import synth
from paper_2605_08632_b200.api import CatLoss

from parity_util import TOL, rel_l2

pytestmark = pytest.mark.gpu


def _sample_blocks(batch, n, rng):
    B = batch.T // batch.K
    blocks = set(rng.choice(B, size=n, replace=False).tolist())
    v = batch.valid.reshape(B, batch.K).bool()
    partly = torch.nonzero((~v).any(1) & v.any(1)).squeeze(1)
    if len(partly):
        blocks.add(int(partly[0])); blocks.add(int(partly[-1]))        # masked blocks on purpose
    if batch.biased.any():
        blocks.add(int(torch.nonzero(batch.biased)[0]) // batch.K)
    blocks = sorted(blocks)
    rows = np.concatenate([np.arange(b * batch.K, (b + 1) * batch.K) for b in blocks])
    return rows


def _check_any_size(batch, out, tol):
    ok = O.effective_valid(batch.labels, batch.valid, batch.V)
    N = int(ok.sum())
    assert out["n_valid"] == N and out["status"] == 0
    w32 = O.cat_weights_f32(out["conf"], ok, batch.K)
    assert out["weight"].tobytes() == w32.tobytes()                      # bit-exact scan, all rows
    ce = -np.log(out["conf"][ok].astype(np.float64))
    loss64 = float((out["weight"][ok].astype(np.float64) * ce).sum() / N)
    assert abs(out["loss"] - loss64) <= 1e-4 * abs(loss64)
    col = np.abs(out["dW"].astype(np.float64).sum(axis=0)).max()
    scale = np.abs(out["dW"].astype(np.float64)).sum(axis=0).max()
    assert col <= 2e-3 * scale, (col, scale)                             # sum_v dz[r, v] = 0
    assert not out["dH"][~ok].any()


def _check_sampled(batch, out, rows, tol):
    H_rows = batch.H[rows]
    sub = synth.Batch(batch.spec, len(rows), batch.K, batch.d, batch.V, H_rows, batch.W, batch.labels[rows],
                      batch.valid[rows], batch.biased[rows])
    fwd = O.cat_forward(sub.H, sub.W, sub.labels, sub.valid, sub.K, row_chunk=256)
    lse_err = np.max(np.abs(out["lse"][rows] - fwd["lse"]) / np.maximum(1.0, np.abs(fwd["lse"])))
    assert lse_err <= tol["lse"], lse_err
    cerr = np.max(np.abs(out["conf"][rows] - fwd["conf"]) / np.maximum(fwd["conf"], 1e-30))
    assert cerr <= tol["conf"], cerr
    werr = np.abs(out["weight"][rows].astype(np.float64) - fwd["weight"])
    assert np.all(werr <= batch.K * tol["conf"] * fwd["weight"] + 1e-37)
    N = int(O.effective_valid(batch.labels, batch.valid, batch.V).sum())
    dH = O.cat_dH_rows(sub.H, sub.W, sub.labels, fwd, np.arange(len(rows)), N)
    assert rel_l2(out["dH"][rows], dH) <= tol["grad"], rel_l2(out["dH"][rows], dH)
    first = np.arange(0, len(rows), batch.K)                              # position-0 rows carry most of the norm;
    later = np.setdiff1d(np.arange(len(rows)), first)                     # check the other positions on their own
    sure = np.exp(np.minimum(fwd["z_label"] - fwd["lse"], 0.0)) > 0.999
    later = later[~sure[later]]
    if np.linalg.norm(dH[later]) > 1e-30:
        assert rel_l2(out["dH"][rows][later], dH[later]) <= 2 * tol["grad"]


def _run(batch, fused):
    dev = torch.device("cuda")
    H, W = batch.H.to(dev), batch.W.to(dev)
    y, valid = batch.labels.to(dev), batch.valid.to(dev)
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K)
    if fused:
        cl.forward_backward(H, W, y, valid)
    else:
        cl.forward(H, W, y, valid)
        cl.backward(H, W, y, valid)
    torch.cuda.synchronize()
    st = cl.fwd_stats()
    out = dict(loss=float(cl.loss.item()), lse=cl.lse.cpu().numpy(), conf=cl.conf.cpu().numpy(),
               weight=cl.weight.cpu().numpy(), dH=cl.dH.float().cpu().numpy(), dW=cl.dW.cpu().numpy(),
               n_valid=st.n_valid, status=st.device_status | (cl.fused_status() if fused else cl.bwd_status()))
    del cl, H, W
    torch.cuda.empty_cache()
    return out


@pytest.mark.parametrize("cfg,n_blocks", [(3, 6), (4, 12), (41, 12), (5, 4)])
def test_full_size_sampled_blocks_and_invariants(cfg, n_blocks):
    batch = synth.make_batch(cfg)
    tol = TOL[torch.bfloat16]
    rows = _sample_blocks(batch, n_blocks, np.random.default_rng(cfg))
    for fused in (True, False):
        out = _run(batch, fused)
        _check_any_size(batch, out, tol)
        _check_sampled(batch, out, rows, tol)
        del out


def test_config2_full_size_whole_forward_and_sampled_dW_rows():
    batch = synth.make_batch(2)
    tol = TOL[torch.bfloat16]
    fwd = O.cat_forward(batch.H, batch.W, batch.labels, batch.valid, batch.K, row_chunk=2048,
                        check_rows_sum_to_one=False)
    rng = np.random.default_rng(2)
    counts = np.bincount(batch.labels.numpy(), minlength=batch.V)
    vocab = np.unique(np.concatenate([rng.choice(batch.V, 200, replace=False), np.argsort(counts)[-28:],
                                      np.nonzero(counts == 0)[0][:28], [0, batch.V - 1]]))
    dW_rows = O.cat_dW_rows(batch.H, batch.W, batch.labels, fwd, vocab)
    rows = _sample_blocks(batch, 8, rng)
    for fused in (True, False):
        out = _run(batch, fused)
        _check_any_size(batch, out, tol)
        _check_sampled(batch, out, rows, tol)
        assert abs(out["loss"] - fwd["loss"]) <= tol["loss"] * fwd["loss"]
        assert np.max(np.abs(out["lse"] - fwd["lse"])) <= tol["lse"] * np.abs(fwd["lse"]).max()
        assert rel_l2(out["dW"][vocab], dW_rows) <= tol["grad"], rel_l2(out["dW"][vocab], dW_rows)
        del out


def test_config2_full_size_distillation_loss_sampled_blocks_and_invariants():
    """cat_kd_loss_fwd_bwd (Eq. 12) at the benchmark's size: a Llama-3.1-8B-shaped target head
    (d_t = 4096) over the T/K + K - 1 sequence positions the batch's blocks refer to."""
    from paper_2605_08632_b200 import binding as B
    batch = synth.make_batch(2)
    ts = synth.make_target_side(batch, d_t=4096)
    tol = TOL[torch.bfloat16]
    beta = 0.1
    dev = torch.device("cuda")
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K)
    cl.kd_forward_backward(batch.H.to(dev), batch.W.to(dev), batch.labels.to(dev), batch.valid.to(dev), ts.Ht.to(dev),
                           ts.Wt.to(dev), ts.block_start, beta)
    torch.cuda.synchronize()
    assert cl.kd_status() == 0 and cl.fwd_stats().device_status == 0
    N = cl.fwd_stats().n_valid
    assert N == batch.T
    conf, weight = cl.conf.cpu().numpy(), cl.weight.cpu().numpy()
    ok = np.ones(batch.T, bool)
    assert weight.tobytes() == O.cat_weights_f32(conf, ok, batch.K).tobytes()        # bit-exact scan, all rows
    dW = cl.dW.cpu().numpy().astype(np.float64)
    assert np.abs(dW.sum(axis=0)).max() <= 2e-3 * np.abs(dW).sum(axis=0).max()       # every dz row sums to zero
    blocks = np.unique(np.r_[np.random.default_rng(12).choice(batch.T // batch.K, 8, replace=False), 0, batch.T // batch.K - 1])
    rows, out, dH_rows = O.cat_kd_rows(batch.H, batch.W, batch.labels, batch.valid, batch.K, ts.Ht, ts.Wt, ts.block_start, beta,
                                       blocks, N)
    assert np.max(np.abs(cl.lse.cpu().numpy()[rows] - out["lse"]) / np.maximum(1.0, np.abs(out["lse"]))) <= tol["lse"]
    assert np.max(np.abs(conf[rows] - out["conf"]) / np.maximum(out["conf"], 1e-30)) <= tol["conf"]
    assert np.all(np.abs(weight[rows] - out["weight"]) <= batch.K * tol["conf"] * out["weight"] + 1e-37)
    assert conf.max() > 0.3 and np.median(conf) < 1e-3                               # the synthetic target spans sure and unsure
    g = cl.dH.float().cpu().numpy()[rows]
    assert rel_l2(g, dH_rows) <= tol["grad"], rel_l2(g, dH_rows)
    later = np.setdiff1d(np.arange(len(rows)), np.arange(0, len(rows), batch.K))
    assert rel_l2(g[later], dH_rows[later]) <= 2 * tol["grad"]
    tot, ce, kd = cl.loss3.cpu().numpy()
    assert abs(tot - (beta * ce + kd)) <= 1e-6 * abs(tot) and kd > 0

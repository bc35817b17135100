"""GPU parity of the entry points beside the CAT objective itself: the fixed position decay
weighting (Table 3 baseline), the per-block acceptance-length estimate (Eq. 8), and the
target-model confidence producer with its draft-row layout (Eq. 9, Eq. 12).  Everything goes
through the C ABI and is compared with the fp64 oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2605_08632_b200 import binding as B
from paper_2605_08632_b200 import synth
from paper_2605_08632_b200.api import CatLoss, TargetConfidence
from parity_util import TOL, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _run(batch, fused, **kw):
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K, dtype=batch.torch_dtype, **kw)
    H, W, y, v = (t.to(DEV) for t in (batch.H, batch.W, batch.labels, batch.valid))
    if fused:
        cl.forward_backward(H, W, y, v)
    else:
        cl.forward(H, W, y, v)
        cl.backward(H, W, y, v)
    torch.cuda.synchronize()
    assert cl.fwd_stats().device_status == 0
    return cl


@pytest.mark.parametrize("fused", [False, True])
@pytest.mark.parametrize("cfg,kw,gamma", [(1, {}, 0.8), (41, dict(T=520, d=256, V=5000), 0.6), (41, dict(T=24 * 5, d=128, V=1024, K=5), 0.8),
                                          (2, dict(T=384, d=512, V=4096), 1.0)])
def test_fixed_decay_matches_oracle(cfg, kw, gamma, fused):
    batch = synth.make_batch(cfg, **kw)
    cl = _run(batch, fused, fixed_decay_gamma=gamma)
    fwd, dH, dW = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, fixed_decay_gamma=gamma)
    tol = TOL[batch.torch_dtype]
    ok = fwd["eff_valid"]
    # weights: bit for bit the binary32 running product of gamma, by position
    w32 = O.fixed_decay_weights_f32(gamma, ok, batch.K)
    assert cl.weight.cpu().numpy().tobytes() == w32.tobytes()
    assert abs(cl.loss.item() - fwd["loss"]) <= tol["loss"] * abs(fwd["loss"])
    # the reported confidences are still the head's own
    cerr = np.abs(cl.conf.cpu().numpy() - fwd["conf"]) / np.maximum(fwd["conf"], 1e-30)
    assert cerr.max() <= tol["conf"]
    assert rel_l2(cl.dH.float().cpu().numpy(), dH) <= tol["grad"]
    assert rel_l2(cl.dW.float().cpu().numpy(), dW) <= tol["grad"]
    # later positions carry real weight here, so check them separately
    T, K = batch.T, batch.K
    g, o = cl.dH.float().cpu().numpy().reshape(T // K, K, -1), dH.reshape(T // K, K, -1)
    for k in range(K):
        nk = np.linalg.norm(o[:, k])
        if nk > 0:
            assert np.linalg.norm(g[:, k] - o[:, k]) / nk <= 2 * tol["grad"], k


def test_fixed_decay_gamma_one_is_uniform_cross_entropy_and_bad_gamma_is_refused():
    batch = synth.make_batch(2, T=256, d=128, V=1000)
    cl = _run(batch, True, fixed_decay_gamma=1.0)
    ce = torch.nn.functional.cross_entropy(batch.H.double() @ batch.W.double().T, batch.labels).item()
    assert abs(cl.loss.item() - ce) <= 1e-3 * ce
    assert np.all(cl.weight.cpu().numpy() == 1.0)
    for bad in (-0.5, float("nan"), float("inf")):
        s = B.make_shape(256, 128, 1000, 8, B.CAT_BF16, weight_mode=B.CAT_WEIGHT_FIXED_DECAY, decay_gamma=bad)
        assert B.cat_loss_workspace_bytes(s, 0) == 0
    s = B.make_shape(256, 128, 1000, 8, B.CAT_BF16, weight_mode=7)
    assert B.cat_loss_workspace_bytes(s, 0) == 0


@pytest.mark.parametrize("cfg,kw", [(41, dict(T=1024, d=256, V=5000)), (41, dict(T=24 * 5, d=128, V=1024, K=5)), (1, {})])
def test_accept_len_estimate(cfg, kw):
    batch = synth.make_batch(cfg, **kw)
    cl = _run(batch, False)
    est = cl.accept_len().cpu().numpy()
    conf, weight = cl.conf.cpu().numpy(), cl.weight.cpu().numpy()
    ref = O.accept_len_estimate(conf, weight, batch.K)          # from the same fp32 conf / weight
    assert est.shape == (batch.T // batch.K,)
    assert np.allclose(est, ref, rtol=1e-5, atol=1e-30)
    # and against the oracle's own forward
    fwd = O.cat_forward(batch.H, batch.W, batch.labels, batch.valid, batch.K)
    ref64 = O.accept_len_estimate(fwd["conf"], fwd["weight"], batch.K)
    assert np.allclose(est, ref64, rtol=batch.K * TOL[batch.torch_dtype]["conf"], atol=1e-30)
    # its mean is what cat_stats reports
    assert abs(cl.fwd_stats().est_accept_len - ref64.mean()) <= 1e-2 * ref64.mean() + 1e-12
    with pytest.raises(B.CatError):
        B.cat_accept_len(B.make_shape(10, 8, 8, 4, B.CAT_BF16), cl.conf, cl.weight, cl.conf)


@pytest.mark.parametrize("cfg,kw,d_t", [(2, dict(T=2048, d=256, V=20000), 384), (41, dict(T=16 * 40, d=128, V=3000, K=16), 128), (1, {}, 64)])
def test_target_confidence_and_window_layout(cfg, kw, d_t):
    batch = synth.make_batch(cfg, **kw)
    ts = synth.make_target_side(batch, d_t=d_t)
    tc = TargetConfidence(ts.L, ts.d_t, batch.V, dtype=batch.torch_dtype)
    tc.forward(ts.Ht.to(DEV), ts.Wt.to(DEV), ts.seq_labels.to(DEV))
    torch.cuda.synchronize()
    assert tc.status() == 0
    conf_o, lse_o = O.target_confidence(ts.Ht, ts.Wt, ts.seq_labels)
    tol = TOL[batch.torch_dtype]
    conf_g = tc.conf_seq.cpu().numpy()
    assert np.max(np.abs(conf_g - conf_o) / np.maximum(conf_o, 1e-30)) <= tol["conf"]
    assert np.max(np.abs(tc.lse_seq.cpu().numpy() - lse_o) / np.maximum(1.0, np.abs(lse_o))) <= tol["lse"]
    assert conf_o.max() > 0.5 and conf_o.min() < 1e-3          # the synthetic target spans sure and unsure
    # layout as draft rows: exact copy of the per-position values
    ce_g = tc.window(ts.block_start.to(DEV), batch.K).cpu().numpy()
    assert ce_g.tobytes() == O.window_confidence(conf_g, ts.block_start, batch.K).astype(np.float32).tobytes()
    # end to end: CAT loss weighted by the target's confidences (the paper's own reading of Eq. 9)
    ce_o = O.window_confidence(conf_o, ts.block_start, batch.K)
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K, dtype=batch.torch_dtype)
    H, W, y, v = (t.to(DEV) for t in (batch.H, batch.W, batch.labels, batch.valid))
    cl.forward_backward(H, W, y, v, conf_ext=torch.from_numpy(ce_g).to(DEV))
    torch.cuda.synchronize()
    fwd, dH, dW = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, conf_ext=ce_o)
    assert abs(cl.loss.item() - fwd["loss"]) <= tol["loss"] * abs(fwd["loss"])
    w_g = cl.weight.cpu().numpy().astype(np.float64)
    assert np.all(np.abs(w_g - fwd["weight"]) <= batch.K * tol["conf"] * fwd["weight"] + 1e-37)
    assert rel_l2(cl.dH.float().cpu().numpy(), dH) <= tol["grad"]
    assert rel_l2(cl.dW.float().cpu().numpy(), dW) <= tol["grad"]


def test_window_edges_and_masked_positions():
    conf = torch.tensor([0.5, 0.25, 0.125, 1.0, 0.75], dtype=torch.float32, device=DEV)
    starts = torch.tensor([-2, 0, 3, 4, 9], dtype=torch.int64, device=DEV)
    out = torch.empty(5 * 3, dtype=torch.float32, device=DEV)
    B.cat_conf_window(conf, 5, starts, 5, 3, out)
    ref = O.window_confidence(conf.cpu().numpy(), starts.cpu().numpy(), 3)
    assert np.array_equal(out.cpu().numpy(), ref.astype(np.float32))
    assert np.array_equal(ref, [1, 1, 0.5, 0.5, 0.25, 0.125, 1.0, 0.75, 1, 0.75, 1, 1, 1, 1, 1])
    # masked / out-of-range labels give confidence 1
    batch = synth.make_batch(2, T=256, d=128, V=1000)
    y = batch.labels.clone(); y[5] = -100; y[9] = 1000
    valid = torch.ones(256, dtype=torch.uint8); valid[17] = 0
    tc = TargetConfidence(256, 128, 1000)
    tc.forward(batch.H.to(DEV), batch.W.to(DEV), y.to(DEV), valid.to(DEV))
    c = tc.conf_seq.cpu().numpy()
    ref, _ = O.target_confidence(batch.H, batch.W, y, valid)
    assert c[5] == c[9] == c[17] == 1.0 and np.allclose(c, ref, rtol=5e-3)


def _golden(name):
    import os
    rows = []
    with open(os.path.join(os.path.dirname(__file__), "golden", name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append([p.strip() for p in line.split("|")])
    return rows


@pytest.mark.parametrize("fused", [False, True])
def test_scan_kernels_on_the_hand_examples(fused):
    """The hand-evaluated instances of Eq. 10 and of the fixed decay (tests/golden/) through the CUDA
    scan (warp-shuffle kernel for K a power of two, per-block kernel otherwise): supplied confidences,
    exact dyadic products, so the weights must match to the bit."""
    dev = "cuda"
    for name, decay in (("eq10_hand_examples.txt", False), ("fixed_decay_hand_examples.txt", True)):
        for K, a, v, w in _golden(name):
            K = int(K)
            valid = torch.tensor([int(x) for x in v.split()], dtype=torch.uint8)
            expect = np.array(w.split(), dtype=np.float32)
            reps = 3                                         # a few blocks, so lanes of several blocks share a warp
            batch = synth.make_batch(2, T=K * reps, d=64, V=256, K=K)
            kw = dict(fixed_decay_gamma=float(a)) if decay else {}
            cl = CatLoss(batch.T, batch.d, batch.V, K, **kw)
            ce = None if decay else torch.tensor([float(x) for x in a.split()] * reps, dtype=torch.float32, device=dev)
            args = (batch.H.to(dev), batch.W.to(dev), batch.labels.to(dev), valid.repeat(reps).to(dev))
            if fused:
                cl.forward_backward(*args, conf_ext=ce)
            else:
                cl.forward(*args, ce)
            torch.cuda.synchronize()
            got = cl.weight.cpu().numpy().reshape(reps, K)
            for r in range(reps):
                assert got[r].tobytes() == expect.tobytes(), (name, K, a, v, got[r], expect)


def test_autograd_module_matches_oracle_and_scales_with_the_upstream_gradient():
    from paper_2605_08632_b200.api import CatLossModule
    batch = synth.make_batch(41, T=512, d=256, V=4000)
    dev = "cuda"
    W = batch.W.to(dev).clone().requires_grad_(True)
    H = batch.H.to(dev).clone().requires_grad_(True)
    head = CatLossModule(W, batch.K)
    loss = head(H, batch.labels.to(dev), batch.valid.to(dev))
    (0.5 * loss).backward()
    torch.cuda.synchronize()
    fwd, dH, dW = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, g=0.5)
    assert abs(loss.item() - fwd["loss"]) <= 1e-3 * fwd["loss"]
    assert H.grad.dtype == torch.bfloat16 and head.weight.grad is not None
    assert rel_l2(H.grad.float().cpu().numpy(), dH) <= 1.2e-2          # one more bf16 rounding from the scaling by 0.5
    assert rel_l2(head.weight.grad.float().cpu().numpy(), dW) <= 1.2e-2


def test_autograd_module_called_twice_with_the_same_shape_before_one_backward():
    """loss = head(H1) + head(H2) with equal T: each term must back-propagate its own gradients."""
    from paper_2605_08632_b200.api import CatLossModule
    b1, b2 = synth.make_batch(41, T=512, d=256, V=4000), synth.make_batch(2, T=512, d=256, V=4000)
    dev = "cuda"
    W = b1.W.to(dev).clone().requires_grad_(True)
    H1, H2 = b1.H.to(dev).clone().requires_grad_(True), b2.H.to(dev).clone().requires_grad_(True)
    head = CatLossModule(W, b1.K)
    loss = head(H1, b1.labels.to(dev), b1.valid.to(dev)) + head(H2, b2.labels.to(dev), b2.valid.to(dev))
    loss.backward()
    torch.cuda.synchronize()
    f1, dH1, dW1 = O.cat_forward_backward(b1.H, b1.W, b1.labels, b1.valid, b1.K)
    f2, dH2, dW2 = O.cat_forward_backward(b2.H, b1.W, b2.labels, b2.valid, b2.K)
    assert abs(loss.item() - (f1["loss"] + f2["loss"])) <= 1e-3 * (f1["loss"] + f2["loss"])
    assert rel_l2(H1.grad.float().cpu().numpy(), dH1) <= 1e-2 and rel_l2(H2.grad.float().cpu().numpy(), dH2) <= 1e-2
    assert rel_l2(head.weight.grad.float().cpu().numpy(), dW1 + dW2) <= 1.2e-2

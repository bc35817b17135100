"""GPU parity of cat_kd_loss_fwd_bwd (Section 3.3, Eq. 12: CAT-weighted cross-entropy plus
distillation from the target head) against the fp64 oracle, through the C ABI.

Tolerances as for the plain CAT loss (bf16 inputs, fp32 accumulation): each loss part within
1e-3 relative (plus 1e-3 of the cross-entropy part as an absolute floor for a distillation part
that is nearly zero), per-tensor gradients within 1e-2 relative L2, weights bit for bit the
binary32 product of the GPU's own confidences."""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2605_08632_b200 import binding as B
from paper_2605_08632_b200 import synth
from paper_2605_08632_b200.api import CatLoss
from parity_util import TOL, rel_l2

pytestmark = pytest.mark.gpu
DEV = "cuda"
T16 = TOL[torch.bfloat16]


def _run_kd(batch, ts_Ht, ts_Wt, starts, beta, slab_mib=0, conf_source=B.CAT_CONF_TARGET, conf_ext=None, g=None, use_valid=True,
            fixed_decay_gamma=None):
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K, dtype=batch.torch_dtype, slab_mib=slab_mib, fixed_decay_gamma=fixed_decay_gamma)
    H, W, y = batch.H.to(DEV), batch.W.to(DEV), batch.labels.to(DEV)
    v = batch.valid.to(DEV) if use_valid else None
    ce = None if conf_ext is None else torch.as_tensor(conf_ext, dtype=torch.float32, device=DEV)
    gl = None if g is None else torch.tensor([g], dtype=torch.float32, device=DEV)
    cl.kd_forward_backward(H, W, y, v, ts_Ht.to(DEV), ts_Wt.to(DEV), starts, beta, conf_source=conf_source, conf_ext=ce, grad_loss=gl)
    torch.cuda.synchronize()
    assert cl.kd_status() == 0 and cl.fwd_stats().device_status == 0
    return dict(loss3=cl.loss3.cpu().numpy().astype(np.float64), lse=cl.lse.cpu().numpy(), conf=cl.conf.cpu().numpy(),
                weight=cl.weight.cpu().numpy(), dH=cl.dH.float().cpu().numpy(), dW=cl.dW.float().cpu().numpy(),
                n_valid=cl.fwd_stats().n_valid, obj=cl)


def _check(gpu, fwd, dH, dW, K, beta, fixed_gamma=None):
    assert gpu["n_valid"] == fwd["n_valid"]
    tot, ce, kd = gpu["loss3"]
    assert abs(ce - fwd["loss_ce"]) <= T16["loss"] * abs(fwd["loss_ce"]) + 1e-12, (ce, fwd["loss_ce"])
    assert abs(kd - fwd["loss_kd"]) <= T16["loss"] * (abs(fwd["loss_kd"]) + abs(fwd["loss_ce"])) + 1e-12, (kd, fwd["loss_kd"])
    assert abs(tot - fwd["loss"]) <= T16["loss"] * (abs(fwd["loss"]) + beta * abs(fwd["loss_ce"])) + 1e-12
    assert abs(tot - (beta * ce + kd)) <= 1e-6 * max(1.0, abs(tot))
    ok = fwd["eff_valid"]
    assert np.max(np.abs(gpu["lse"] - fwd["lse"]) / np.maximum(1.0, np.abs(fwd["lse"]))) <= T16["lse"]
    cerr = np.abs(gpu["conf"] - fwd["conf"]) / np.maximum(np.abs(fwd["conf"]), 1e-30)
    assert cerr.max() <= T16["conf"], cerr.max()
    if fixed_gamma is None:
        w32 = O.cat_weights_f32(gpu["conf"].astype(np.float32), ok, K)
    else:
        w32 = O.fixed_decay_weights_f32(fixed_gamma, ok, K)
    assert gpu["weight"].tobytes() == w32.tobytes()
    assert rel_l2(gpu["dH"], dH) <= T16["grad"], rel_l2(gpu["dH"], dH)
    assert rel_l2(gpu["dW"], dW) <= T16["grad"], rel_l2(gpu["dW"], dW)
    assert not gpu["dH"][~ok].any()
    T = dH.shape[0]
    gH, oH = gpu["dH"].reshape(T // K, K, -1), dH.reshape(T // K, K, -1)
    top = np.linalg.norm(oH[:, 0])
    for k in range(K):
        nk = np.linalg.norm(oH[:, k])
        if nk > 1e-25 * top and nk > 1e-30:
            assert np.linalg.norm(gH[:, k] - oH[:, k]) / nk <= 2 * T16["grad"], k


@pytest.mark.parametrize("cfg,kw,d_t,slab_mib", [
    (2, dict(T=512, d=256, V=5000), 384, 0),
    (41, dict(T=1000, d=200, V=5000), 136, 1),           # several row slabs, masked rows, ragged everything
    (41, dict(T=24 * 5, d=128, V=1024, K=5), 128, 1),    # block length that is not a power of two
    (3, dict(T=16 * 48, d=128, V=3000), 256, 0),         # K = 16
])
def test_kd_matches_oracle_with_target_confidences(cfg, kw, d_t, slab_mib):
    batch = synth.make_batch(cfg, **kw)
    ts = synth.make_target_side(batch, d_t=d_t)
    beta = 0.1
    gpu = _run_kd(batch, ts.Ht, ts.Wt, ts.block_start, beta, slab_mib=slab_mib)
    fwd, dH, dW = O.cat_kd_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, ts.Ht, ts.Wt, ts.block_start, beta)
    assert fwd["conf"][fwd["eff_valid"]].max() > 0.3       # the synthetic target is sure of some labels: real weights downstream
    _check(gpu, fwd, dH, dW, batch.K, beta)


def test_kd_other_confidence_sources_scale_and_fixed_decay():
    batch = synth.make_batch(41, T=768, d=256, V=4000)
    ts = synth.make_target_side(batch, d_t=192)
    args = (batch.H, batch.W, batch.labels, batch.valid, batch.K, ts.Ht, ts.Wt, ts.block_start)
    # the draft's own confidence
    gpu = _run_kd(batch, ts.Ht, ts.Wt, ts.block_start, 0.5, conf_source=B.CAT_CONF_DRAFT, g=0.25)
    fwd, dH, dW = O.cat_kd_forward_backward(*args, 0.5, conf_source="draft", g=0.25)
    _check(gpu, fwd, dH, dW, batch.K, 0.5)
    # confidences supplied by the caller
    ce = np.random.default_rng(3).random(batch.T).astype(np.float32)
    gpu = _run_kd(batch, ts.Ht, ts.Wt, ts.block_start, 0.1, conf_ext=ce, use_valid=False)
    fwd, dH, dW = O.cat_kd_forward_backward(batch.H, batch.W, batch.labels, None, batch.K, ts.Ht, ts.Wt, ts.block_start, 0.1, conf_ext=ce)
    _check(gpu, fwd, dH, dW, batch.K, 0.1)
    # beta = 0: distillation only;  fixed position decay instead of CAT weights
    gpu = _run_kd(batch, ts.Ht, ts.Wt, ts.block_start, 0.0, fixed_decay_gamma=0.8)
    fwd, dH, dW = O.cat_kd_forward_backward(*args, 0.0, fixed_decay_gamma=0.8)
    _check(gpu, fwd, dH, dW, batch.K, 0.0, fixed_gamma=0.8)


def test_kd_rows_without_a_target_position_are_invalid():
    batch = synth.make_batch(2, T=512, d=128, V=3000)
    ts = synth.make_target_side(batch, d_t=128)
    starts = ts.block_start.clone() + 3          # the last blocks now run past the end of the sequence
    starts[:2] = torch.tensor([-2, -1])          # and the first two start before it
    gpu = _run_kd(batch, ts.Ht, ts.Wt, starts, 0.1)
    fwd, dH, dW = O.cat_kd_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, ts.Ht, ts.Wt, starts, 0.1)
    assert fwd["n_valid"] < batch.T and not fwd["eff_valid"][0] and fwd["eff_valid"][2]
    _check(gpu, fwd, dH, dW, batch.K, 0.1)


def test_kd_with_the_draft_as_its_own_target_is_beta_times_cat():
    batch = synth.make_batch(41, T=512, d=128, V=3000)
    starts = torch.arange(batch.T // batch.K, dtype=torch.int64) * batch.K      # every draft row its own target row
    ce = np.full(batch.T, 0.5, np.float32)
    gpu = _run_kd(batch, batch.H, batch.W, starts, 0.3, conf_ext=ce)
    cat, dH, dW = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid, batch.K, conf_ext=ce, g=0.3)
    tot, cel, kdl = gpu["loss3"]
    assert abs(kdl) <= 1e-3 * cat["loss"] and abs(cel - cat["loss"]) <= 1e-3 * cat["loss"]
    assert rel_l2(gpu["dH"], dH) <= 1e-2 and rel_l2(gpu["dW"], dW) <= 1e-2


def test_kd_argument_errors_and_determinism():
    batch = synth.make_batch(2, T=256, d=128, V=2000)
    ts = synth.make_target_side(batch, d_t=128)
    s = B.make_shape(256, 128, 2000, 8, B.CAT_BF16)
    desc = B.make_kd_desc(ts.L, 128, 0.1)
    assert B.cat_kd_workspace_bytes(s, desc, ts.block_start) > B.cat_loss_workspace_bytes(s, 2)
    unsorted = ts.block_start.clone(); unsorted[3] = 100
    assert B.cat_kd_workspace_bytes(s, desc, unsorted) == 0
    assert B.cat_kd_workspace_bytes(B.make_shape(256, 128, 2000, 8, B.CAT_F32), desc, ts.block_start) == 0
    assert B.cat_kd_workspace_bytes(s, B.make_kd_desc(ts.L, 132, 0.1), ts.block_start) == 0
    assert B.cat_kd_workspace_bytes(s, B.make_kd_desc(ts.L, 128, -1.0), ts.block_start) == 0
    cl = CatLoss(256, 128, 2000, 8)
    with pytest.raises(B.CatError) as e:
        cl.loss3 = torch.zeros(3, device=DEV)
        ws = torch.empty(1 << 20, dtype=torch.uint8, device=DEV)
        B.cat_kd_loss_fwd_bwd(s, desc, batch.H.to(DEV), batch.W.to(DEV), batch.labels.to(DEV), None, ts.Ht.to(DEV), ts.Wt.to(DEV),
                              unsorted, None, None, cl.loss3, cl.lse, cl.conf, cl.weight, cl.stats, cl.dH, cl.dW, False, ws)
    assert e.value.code == -2
    a = _run_kd(batch, ts.Ht, ts.Wt, ts.block_start, 0.1)
    b = _run_kd(batch, ts.Ht, ts.Wt, ts.block_start, 0.1)
    for key in ("lse", "conf", "weight", "dH", "dW"):
        assert a[key].tobytes() == b[key].tobytes(), key
    assert a["loss3"].tobytes() == b["loss3"].tobytes()

"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI, run the
oracle on the same seeded batch, and compare element by element with the stated tolerances.

Tolerances (bf16 inputs, fp32 accumulation): loss relative error <= 1e-3, per-tensor gradient
relative L2 error <= 1e-2.  fp32 config: loss 1e-5, gradients 1e-4, confidences 1e-5.
The CAT weight vector must equal, bit for bit, the binary32 left-to-right product of the
GPU's own confidences (the bit-exact claim), and agree with the fp64 oracle's weights within
rounding; products that underflow binary32 (~V^-k for k large) are compared with an absolute
floor.
"""
import numpy as np
import torch

from oracle import cat_oracle as O
from paper_2605_08632_b200.api import CatLoss

# Per-position-class dH checks allow this multiple of the per-tensor gradient tolerance: a class holds
# 1/K of the rows and, past position 0, gradients ~V^-k of the tensor's norm, so the bf16 rounding of
# dz and dH that averages out over the tensor shows more in one class.
POSITION_FACTOR = 2.0

TOL = {
    torch.bfloat16: dict(loss=1e-3, grad=1e-2, lse=2e-3, conf=5e-3),
    torch.float32: dict(loss=1e-5, grad=1e-4, lse=1e-5, conf=1e-5),
}


def rel_l2(a, b):
    a = np.asarray(a, np.float64); b = np.asarray(b, np.float64)
    den = np.linalg.norm(b)
    return float(np.linalg.norm(a - b) / den) if den > 0 else float(np.linalg.norm(a))


def run_gpu(batch, slab_mib=0, g=None, conf_ext=None, dW_dtype=torch.float32, use_valid=True, accumulate_into=None):
    dev = torch.device("cuda")
    H, W = batch.H.to(dev), batch.W.to(dev)
    labels = batch.labels.to(dev)
    valid = batch.valid.to(dev) if use_valid else None
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K, dtype=batch.torch_dtype, dW_dtype=dW_dtype, slab_mib=slab_mib)
    ce = None if conf_ext is None else torch.as_tensor(conf_ext, dtype=torch.float32, device=dev)
    gl = None if g is None else torch.tensor([g], dtype=torch.float32, device=dev)
    cl.forward(H, W, labels, valid, ce)
    acc = False
    if accumulate_into is not None:
        cl.dW.copy_(torch.as_tensor(accumulate_into, device=dev).to(dW_dtype))
        acc = True
    cl.backward(H, W, labels, valid, gl, accumulate_dW=acc)
    torch.cuda.synchronize()
    st = cl.fwd_stats()
    out = dict(loss=float(cl.loss.item()), lse=cl.lse.cpu().numpy(), conf=cl.conf.cpu().numpy(),
               weight=cl.weight.cpu().numpy(), dH=cl.dH.float().cpu().numpy(), dW=cl.dW.float().cpu().numpy(),
               stats=st, bwd_status=cl.bwd_status(), obj=cl)
    return out


def run_gpu_fused(batch, slab_mib=0, g=None, conf_ext=None, dW_dtype=torch.float32, use_valid=True, accumulate_into=None):
    """Same outputs as run_gpu, through the single cat_loss_fwd_bwd call."""
    dev = torch.device("cuda")
    H, W = batch.H.to(dev), batch.W.to(dev)
    labels = batch.labels.to(dev)
    valid = batch.valid.to(dev) if use_valid else None
    cl = CatLoss(batch.T, batch.d, batch.V, batch.K, dtype=batch.torch_dtype, dW_dtype=dW_dtype, slab_mib=slab_mib)
    ce = None if conf_ext is None else torch.as_tensor(conf_ext, dtype=torch.float32, device=dev)
    gl = None if g is None else torch.tensor([g], dtype=torch.float32, device=dev)
    acc = False
    if accumulate_into is not None:
        cl.dW.copy_(torch.as_tensor(accumulate_into, device=dev).to(dW_dtype))
        acc = True
    cl.forward_backward(H, W, labels, valid, ce, gl, accumulate_dW=acc)
    torch.cuda.synchronize()
    return dict(loss=float(cl.loss.item()), lse=cl.lse.cpu().numpy(), conf=cl.conf.cpu().numpy(),
                weight=cl.weight.cpu().numpy(), dH=cl.dH.float().cpu().numpy(), dW=cl.dW.float().cpu().numpy(),
                stats=cl.fwd_stats(), bwd_status=cl.fused_status(), obj=cl)


def run_oracle(batch, g=1.0, conf_ext=None, use_valid=True):
    fwd, dH, dW = O.cat_forward_backward(batch.H, batch.W, batch.labels, batch.valid if use_valid else None, batch.K,
                                         conf_ext=conf_ext, g=g)
    return fwd, dH, dW


def check_forward(gpu, fwd, K, dtype, V):
    tol = TOL[dtype]
    ok = fwd["eff_valid"]
    assert gpu["stats"].device_status == 0
    assert gpu["stats"].n_valid == fwd["n_valid"]
    assert abs(gpu["loss"] - fwd["loss"]) <= tol["loss"] * abs(fwd["loss"]) + 1e-12, (gpu["loss"], fwd["loss"])
    assert np.max(np.abs(gpu["lse"] - fwd["lse"]) / np.maximum(1.0, np.abs(fwd["lse"]))) <= tol["lse"]
    # confidences: relative, with an absolute floor far below anything that matters
    cerr = np.abs(gpu["conf"] - fwd["conf"]) / np.maximum(np.abs(fwd["conf"]), 1e-30)
    assert np.max(cerr) <= tol["conf"], np.max(cerr)
    assert np.all(gpu["conf"][~ok] == 1.0)
    # bit-exact: weights are the binary32 left-to-right product of the GPU's own confidences
    w32 = O.cat_weights_f32(gpu["conf"].astype(np.float32), ok, K)
    assert gpu["weight"].tobytes() == w32.tobytes()
    # and they agree with the fp64 oracle's weights (K-1 factors, each within tol["conf"])
    werr = np.abs(gpu["weight"].astype(np.float64) - fwd["weight"])
    assert np.all(werr <= K * tol["conf"] * fwd["weight"] + 1e-37), np.max(werr / np.maximum(fwd["weight"], 1e-37))
    assert np.all(gpu["weight"][~ok] == 0.0)


def check_dH_rows_by_position(gH, oH, fwd, K, W_row_norm_max, N, g, tol_grad):
    """dH compared separately for every position in the draft block (the loss is dominated by
    position 0, so a per-tensor norm alone would hide a wrong scan), `gH` / `oH` / `fwd` covering the
    same whole blocks.

    Rows with label probability <= 0.999: relative L2 over the rows of one position class,
    <= POSITION_FACTOR * tol_grad.
    Near-certain rows (p_y > 0.999) are bounded one by one instead of being left out.  Their gradient is
    c_r (sum_v p_v W_v - W_y), c_r = g w_r / N, which nearly cancels: what the CUDA path can resolve of
    1 - p_y is limited by binary32 -- the backward receives lse as a float, and z_y, lse near 16 have
    an ulp of 1.9e-6.  An absolute error eps in the exponent z_v - lse scales every p_v by (1 + eps), i.e.
    moves the row's gradient by at most c_r * eps * max_v |W_v|.  With eps_r = 2^-20 * max(1, |lse_r|, |z_y|)
    (eight binary32 ulps for rounding lse, the logit accumulation and exp/log) the bound per row is
        |dH_gpu[r] - dH_oracle[r]| <= POSITION_FACTOR * tol_grad * |dH_oracle[r]| + c_r * eps_r * max_v |W_v| + floor,
    floor = sqrt(d) * 2^-126: entries below the smallest normal binary32 / bfloat16 number lose their bits.
    A dropped one-hot or a wrong sign on such a row is an error of c_r * |W_y|, five orders above it."""
    T = oH.shape[0]
    p_label = np.exp(np.minimum(fwd["z_label"] - fwd["lse"], 0.0))
    sure = (p_label > 0.999) & fwd["eff_valid"]
    keep = (~sure).reshape(T // K, K)
    g3, o3 = gH.reshape(T // K, K, -1), oH.reshape(T // K, K, -1)
    top = np.linalg.norm(o3[:, 0])
    for k in range(K):
        nk = np.linalg.norm(o3[keep[:, k], k])
        if nk > 1e-30 and nk > 1e-25 * top:
            e = np.linalg.norm(g3[keep[:, k], k] - o3[keep[:, k], k]) / nk
            assert e <= POSITION_FACTOR * tol_grad, (k, e)
    rows = np.nonzero(sure)[0]
    if len(rows):
        c = abs(g) * fwd["weight"][rows] / max(N, 1)
        eps = 2.0 ** -20 * np.maximum(1.0, np.maximum(np.abs(fwd["lse"][rows]), np.abs(fwd["z_label"][rows])))
        err = np.linalg.norm(gH[rows].astype(np.float64) - oH[rows], axis=1)
        bound = (POSITION_FACTOR * tol_grad * np.linalg.norm(oH[rows], axis=1) + c * eps * W_row_norm_max
                 + np.sqrt(oH.shape[1]) * 2.0 ** -126)
        worst = int(np.argmax(err - bound))
        assert np.all(err <= bound), (int(rows[worst]), float(err[worst]), float(bound[worst]))
    return int(len(rows))


def check_backward(gpu, fwd, dH, dW, K, dtype, per_position=True, W=None, g=1.0):
    tol = TOL[dtype]
    assert gpu["bwd_status"] == 0
    assert rel_l2(gpu["dH"], dH) <= tol["grad"], rel_l2(gpu["dH"], dH)
    assert rel_l2(gpu["dW"], dW) <= tol["grad"], rel_l2(gpu["dW"], dW)
    ok = fwd["eff_valid"]
    assert not gpu["dH"][~ok].any()
    if per_position:
        if W is None:
            raise ValueError("the per-position check needs W (row norms bound the near-certain rows)")
        Wd = W.double().numpy() if hasattr(W, "double") else np.asarray(W, np.float64)
        check_dH_rows_by_position(gpu["dH"], dH, fwd, K, float(np.sqrt((Wd * Wd).sum(axis=1).max())), fwd["n_valid"], g,
                                  tol["grad"])

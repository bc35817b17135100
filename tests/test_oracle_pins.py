"""Pins for the fp64 oracle: it is checked against what the paper's formulas and plain
mathematics fix, never against itself and never against the CUDA path.

Each test names the equation it pins.  A dropped term, a wrong sign or index, an inclusive
instead of exclusive product, a gradient through the weights, or a wrong normaliser fails
at least one of them.
"""
import math
import os

import numpy as np
import pytest
import torch

from oracle import cat_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_problem(seed, T, d, V, scale=0.3, masked=False):
    rng = np.random.default_rng(seed)
    H = rng.standard_normal((T, d))
    W = rng.standard_normal((V, d)) * scale
    y = rng.integers(0, V, size=T)
    valid = np.ones(T, dtype=np.uint8)
    if masked:
        valid[rng.random(T) < 0.25] = 0
    return H, W, y, valid


# ---------------------------------------------------------------- Eq. 10: hand examples
def _read_hand_examples():
    out = []
    with open(os.path.join(GOLDEN, "eq10_hand_examples.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, c, v, w = [p.strip() for p in line.split("|")]
            out.append((int(k), np.array(c.split(), float), np.array(v.split(), int), np.array(w.split(), float)))
    return out


@pytest.mark.parametrize("K,c,v,w", _read_hand_examples())
def test_eq10_hand_examples(K, c, v, w):
    assert np.array_equal(O.cat_weights(c, v.astype(bool), K), w)
    assert np.array_equal(O.cat_weights_f32(c.astype(np.float32), v.astype(bool), K), w.astype(np.float32))


def test_eq10_first_weight_is_one_and_recurrence():
    rng = np.random.default_rng(1)
    K, B = 16, 37
    c = rng.random(B * K)
    ok = np.ones(B * K, bool)
    w = O.cat_weights(c, ok, K).reshape(B, K)
    cc = c.reshape(B, K)
    assert np.all(w[:, 0] == 1.0)                                   # s_0 := 1
    assert np.allclose(w[:, 1:], w[:, :-1] * cc[:, :-1], rtol=0, atol=0)  # s_{k+1} = s_k c_k
    assert np.all(np.diff(w, axis=1) <= 0) and np.all((w >= 0) & (w <= 1))
    # the weight of row k must not contain c_k itself (exclusive product)
    c2 = cc.copy(); c2[:, 5] = 0.123
    w2 = O.cat_weights(c2.reshape(-1), ok, K).reshape(B, K)
    assert np.array_equal(w2[:, :6], w[:, :6]) and not np.array_equal(w2[:, 6], w[:, 6])


def test_eq6_eq8_acceptance_length_identity():
    # sum_k s_k c_k == sum_k prod_{j<=k} c_j  (Eq. 6 rewritten as Eq. 8)
    rng = np.random.default_rng(2)
    K = 8
    c = rng.random(5 * K)
    w = O.cat_weights(c, np.ones_like(c, bool), K).reshape(5, K)
    lhs = (w * c.reshape(5, K)).sum(axis=1)
    rhs = np.cumprod(c.reshape(5, K), axis=1).sum(axis=1)
    assert np.allclose(lhs, rhs, rtol=1e-14)


def test_constant_confidence_is_fixed_decay():
    # with c == gamma, Eq. 10 gives s_k = gamma^k: the fixed position decay the paper ablates against
    H, W, y, valid = _rand_problem(3, 4 * 8, 8, 32)
    for gamma in (1.0, 0.8, 0.6):
        fwd = O.cat_forward(H, W, y, valid, 8, conf_ext=np.full(32, gamma))
        expect = np.tile(gamma ** np.arange(8), 4)
        assert np.allclose(fwd["weight"], expect, rtol=1e-14)
        ce = fwd["lse"] - fwd["z_label"]
        assert math.isclose(fwd["loss"], float((expect * ce).mean()), rel_tol=1e-13)


# ---------------------------------------------------------------- fixed position decay (Table 3 baseline)
def _read_decay_examples():
    out = []
    with open(os.path.join(GOLDEN, "fixed_decay_hand_examples.txt")) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, g, v, w = [p.strip() for p in line.split("|")]
            out.append((int(k), float(g), np.array(v.split(), int), np.array(w.split(), float)))
    return out


@pytest.mark.parametrize("K,gamma,v,w", _read_decay_examples())
def test_fixed_decay_hand_examples(K, gamma, v, w):
    assert np.array_equal(O.fixed_decay_weights(gamma, v.astype(bool), K), w)
    assert np.array_equal(O.fixed_decay_weights_f32(gamma, v.astype(bool), K), w.astype(np.float32))


def test_fixed_decay_matches_closed_form_and_the_constant_confidence_case():
    H, W, y, valid = _rand_problem(13, 5 * 8, 8, 32)
    for gamma in (1.0, 0.8, 0.6):                       # the three rates of Table 3
        fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, 8, fixed_decay_gamma=gamma)
        assert np.allclose(fwd["weight"].reshape(-1, 8), gamma ** np.arange(8), rtol=1e-14)
        # with every row valid it is CAT with all confidences equal to gamma
        ref, dH2, dW2 = O.cat_forward_backward(H, W, y, valid, 8, conf_ext=np.full(40, gamma))
        assert math.isclose(fwd["loss"], ref["loss"], rel_tol=1e-13)
        assert np.allclose(dH, dH2, rtol=1e-12, atol=1e-18) and np.allclose(dW, dW2, rtol=1e-12, atol=1e-18)
    # gamma = 1 is the uniform loss of Eq. 5
    one = O.cat_forward(H, W, y, valid, 8, fixed_decay_gamma=1.0)
    loss_t, _, _ = _torch_ce(H, W, y, valid, 40)
    assert math.isclose(one["loss"], loss_t, rel_tol=1e-12)
    # the model's own confidences are still reported, and play no part in the weights
    assert np.allclose(one["conf"], np.exp(one["z_label"] - one["lse"]), rtol=1e-14)


def test_fixed_decay_counts_positions_not_valid_rows():
    ok = np.array([1, 0, 0, 1, 1, 1, 0, 1], bool)
    w = O.fixed_decay_weights(0.5, ok, 4).reshape(2, 4)
    assert np.array_equal(w, [[1, 0, 0, 0.125], [1, 0.5, 0, 0.125]])
    # CAT with constant confidence skips masked rows instead: the two differ exactly there
    w_cat = O.cat_weights(np.full(8, 0.5), ok, 4).reshape(2, 4)
    assert np.array_equal(w_cat, [[1, 0, 0, 0.5], [1, 0.5, 0, 0.25]])


# ---------------------------------------------------------------- Eq. 8 estimate per block
def test_accept_len_estimate_closed_forms():
    K = 8
    # constant confidence c: sum_k c^k * c = c (1 - c^K) / (1 - c)
    for c in (0.9, 0.5, 0.1):
        conf = np.full(3 * K, c)
        w = O.cat_weights(conf, np.ones(3 * K, bool), K)
        est = O.accept_len_estimate(conf, w, K)
        assert np.allclose(est, c * (1 - c ** K) / (1 - c), rtol=1e-13)
    # certain drafter: every token accepted, length K;  first token never accepted: length 0
    ones = np.ones(K)
    assert O.accept_len_estimate(ones, O.cat_weights(ones, ones.astype(bool), K), K)[0] == K
    c0 = np.array([0.0] + [0.7] * (K - 1))
    assert O.accept_len_estimate(c0, O.cat_weights(c0, np.ones(K, bool), K), K)[0] == 0.0
    # Eq. 3 by brute force: E[L] = sum over acceptance patterns of (prefix length * probability)
    rng = np.random.default_rng(5)
    c = rng.random(4)
    brute = 0.0
    for bits in range(16):
        acc = [(bits >> k) & 1 for k in range(4)]
        prob = np.prod([c[k] if acc[k] else 1 - c[k] for k in range(4)])
        length = 0
        while length < 4 and acc[length]:
            length += 1
        brute += prob * length
    est = O.accept_len_estimate(c, O.cat_weights(c, np.ones(4, bool), 4), 4)[0]
    assert math.isclose(est, brute, rel_tol=1e-13)


# ---------------------------------------------------------------- Eq. 9 with a target head, Eq. 12 layout
def test_target_confidence_is_softmax_probability_of_the_label():
    rng = np.random.default_rng(21)
    L, dt, V = 19, 6, 11
    Ht, Wt = rng.standard_normal((L, dt)), rng.standard_normal((V, dt))
    y = rng.integers(0, V, L)
    y[3] = -100
    conf, lse = O.target_confidence(Ht, Wt, y)
    p = torch.softmax(torch.tensor(Ht @ Wt.T), dim=1).numpy()
    for i in range(L):
        assert math.isclose(conf[i], 1.0 if i == 3 else p[i, y[i]], rel_tol=1e-13)
    assert np.allclose(lse, torch.logsumexp(torch.tensor(Ht @ Wt.T), dim=1).numpy(), rtol=1e-14)
    # Wt = 0: every token has probability 1/V
    c0, l0 = O.target_confidence(Ht, np.zeros((V, dt)), y)
    assert np.allclose(np.delete(c0, 3), 1.0 / V, rtol=1e-14) and np.allclose(l0, math.log(V), rtol=1e-14)


def test_window_confidence_gives_the_sliding_product_of_eq12():
    # a sequence of L positions with confidences c_i; the block that starts at position n holds
    # c_n..c_{n+K-1}, so Eq. 10 on it gives s_{n,k} = prod_{j<k} c_{n+j}: a window sliding with n
    rng = np.random.default_rng(22)
    L, K = 12, 4
    c = rng.random(L)
    starts = np.arange(0, L)                 # one block per prefix position
    ce = O.window_confidence(c, starts, K)
    assert ce.shape == (L * K,)
    ok = np.array([[n + k < L for k in range(K)] for n in starts]).reshape(-1)   # Eq. 12: n <= N - k
    w = O.cat_weights(ce, ok, K).reshape(L, K)
    for n in range(L):
        for k in range(K):
            if n + k < L:
                assert ce[n * K + k] == c[n + k]
                assert math.isclose(w[n, k], float(np.prod(c[n:n + k])), rel_tol=1e-14)
            else:
                assert ce[n * K + k] == 1.0 and w[n, k] == 0.0
    # the same target position carries the same confidence in every block that contains it
    assert ce[0 * K + 3] == ce[1 * K + 2] == ce[2 * K + 1] == ce[3 * K + 0] == c[3]
    # a start before the sequence or past its end reads as 1
    assert np.array_equal(O.window_confidence(c, np.array([-2, L - 1]), K), [1, 1, c[0], c[1], c[L - 1], 1, 1, 1])


# ---------------------------------------------------------------- Eq. 5 / Eq. 11 degenerate cases
def _torch_ce(H, W, y, valid, reduction_n):
    Ht = torch.tensor(H, dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(W, dtype=torch.float64, requires_grad=True)
    yt = torch.tensor(np.where(valid.astype(bool), y, -100))
    loss = torch.nn.functional.cross_entropy(Ht @ Wt.T, yt, ignore_index=-100, reduction="sum") / reduction_n
    loss.backward()
    return loss.item(), Ht.grad.numpy(), Wt.grad.numpy()


@pytest.mark.parametrize("masked", [False, True])
def test_unit_confidence_reduces_to_mean_cross_entropy(masked):
    # all prefix confidences 1 => s == 1 => Eq. 11 is the uniform PARD loss of Eq. 5
    H, W, y, valid = _rand_problem(4, 6 * 4, 8, 32, masked=masked)
    fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, 4, conf_ext=np.ones(24), g=1.0)
    n = int(valid.sum())
    loss_t, dH_t, dW_t = _torch_ce(H, W, y, valid, n)
    assert fwd["n_valid"] == n
    assert np.array_equal(fwd["weight"], valid.astype(float))
    assert math.isclose(fwd["loss"], loss_t, rel_tol=1e-12)
    assert np.allclose(dH, dH_t, rtol=1e-10, atol=1e-14)
    assert np.allclose(dW, dW_t, rtol=1e-10, atol=1e-14)


def test_K1_is_plain_cross_entropy_in_self_confidence_mode():
    # K = 1: every row is position 0, s_0 := 1 whatever the confidences are
    H, W, y, valid = _rand_problem(5, 20, 8, 32, masked=True)
    fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, 1, g=0.7)
    loss_t, dH_t, dW_t = _torch_ce(H, W, y, valid, int(valid.sum()))
    assert math.isclose(fwd["loss"], loss_t, rel_tol=1e-12)
    assert np.allclose(dH, 0.7 * dH_t, rtol=1e-10, atol=1e-14)
    assert np.allclose(dW, 0.7 * dW_t, rtol=1e-10, atol=1e-14)


def test_W_zero_closed_form():
    # W = 0: p == 1/V, c = 1/V, s_k = V^-k, loss = (ln V / K) (1 - V^-K)/(1 - 1/V); dH = 0
    T, d, V, K = 24, 8, 32, 4
    H, _, y, valid = _rand_problem(6, T, d, V)
    W = np.zeros((V, d))
    fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, K)
    assert np.allclose(fwd["conf"], 1.0 / V, rtol=1e-14)
    assert np.allclose(fwd["weight"].reshape(-1, K), (1.0 / V) ** np.arange(K), rtol=1e-13)
    closed = math.log(V) / K * (1 - V ** (-K)) / (1 - 1 / V)
    assert math.isclose(fwd["loss"], closed, rel_tol=1e-13)
    assert np.all(dH == 0)
    w = fwd["weight"]
    expect_dW = np.zeros((V, d))
    for r in range(T):
        for v in range(V):
            expect_dW[v] += (w[r] / T) * (1.0 / V - (1.0 if v == y[r] else 0.0)) * H[r]
    assert np.allclose(dW, expect_dW, rtol=1e-12, atol=1e-16)


# ---------------------------------------------------------------- brute force, pure Python
def _brute_force(H, W, y, valid, K, g):
    """Eq. 9-11 and the frozen-weight gradient in pure Python lists and math.exp, no max-subtraction."""
    T, d, V = len(H), len(H[0]), len(W)
    p = []
    for r in range(T):
        z = [sum(H[r][i] * W[v][i] for i in range(d)) for v in range(V)]
        e = [math.exp(t) for t in z]
        s = sum(e)
        p.append([t / s for t in e])
    ok = [bool(valid[r]) and 0 <= y[r] < V for r in range(T)]
    N = sum(ok)
    w = [0.0] * T
    for b in range(T // K):
        s = 1.0
        for k in range(K):
            r = b * K + k
            if ok[r]:
                w[r] = s
                s *= p[r][y[r]]
    loss = sum(-w[r] * math.log(p[r][y[r]]) for r in range(T) if ok[r]) / N
    dH = [[0.0] * d for _ in range(T)]
    dW = [[0.0] * d for _ in range(V)]
    for r in range(T):
        if not ok[r]:
            continue
        for v in range(V):
            dz = g * w[r] / N * (p[r][v] - (1.0 if v == y[r] else 0.0))
            for i in range(d):
                dH[r][i] += dz * W[v][i]
                dW[v][i] += dz * H[r][i]
    return loss, w, dH, dW


def test_brute_force_tiny_with_mask_and_bad_label():
    T, d, V, K = 12, 4, 7, 4
    H, W, y, valid = _rand_problem(7, T, d, V, scale=0.8, masked=True)
    y = y.copy(); y[3] = V + 2; valid[3] = 1; valid[0] = 1; valid[1] = 1   # out-of-range label on a valid row
    fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, K, g=1.3)
    loss_b, w_b, dH_b, dW_b = _brute_force(H.tolist(), W.tolist(), y.tolist(), valid.tolist(), K, 1.3)
    assert math.isclose(fwd["loss"], loss_b, rel_tol=1e-12)
    assert np.allclose(fwd["weight"], w_b, rtol=1e-12)
    assert np.allclose(dH, dH_b, rtol=1e-10, atol=1e-15)
    assert np.allclose(dW, dW_b, rtol=1e-10, atol=1e-15)
    assert fwd["weight"][3] == 0 and np.all(dH[3] == 0)


# ---------------------------------------------------------------- gradients: stop-gradient on s
def _loss_with_weights(H, W, y, valid, K, w_fixed):
    fwd = O.cat_forward(H, W, y, valid, K)
    ce = fwd["lse"] - fwd["z_label"]
    return float((w_fixed * np.where(fwd["eff_valid"], ce, 0.0)).sum() / fwd["n_valid"])


def test_finite_differences_with_frozen_weights_and_converse():
    T, d, V, K = 8, 8, 32, 4
    H, W, y, valid = _rand_problem(8, T, d, V, scale=0.5)
    H[:, :] += 2.0 * W[y]            # push confidences up so later positions carry weight
    valid[5] = 0
    fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, K)
    w0 = fwd["weight"]
    assert w0.reshape(-1, K)[:, 1:].max() > 1e-2
    eps = 1e-6
    rng = np.random.default_rng(9)
    worst = 0.0
    moved = 0.0
    for _ in range(40):
        if rng.random() < 0.5:
            r, i = rng.integers(T), rng.integers(d)
            def bump(s, r=r, i=i):
                Hp = H.copy(); Hp[r, i] += s; return Hp, W
            ana = dH[r, i]
        else:
            v, i = rng.integers(V), rng.integers(d)
            def bump(s, v=v, i=i):
                Wp = W.copy(); Wp[v, i] += s; return H, Wp
            ana = dW[v, i]
        Hp, Wp = bump(eps); Hm, Wm = bump(-eps)
        fd_frozen = (_loss_with_weights(Hp, Wp, y, valid, K, w0) - _loss_with_weights(Hm, Wm, y, valid, K, w0)) / (2 * eps)
        fd_free = (O.cat_forward(Hp, Wp, y, valid, K)["loss"] - O.cat_forward(Hm, Wm, y, valid, K)["loss"]) / (2 * eps)
        # central differences carry ~1e-10 absolute rounding noise (loss ~ 1, eps 1e-6)
        worst = max(worst, abs(fd_frozen - ana) / (abs(ana) + 1e-3))
        moved = max(moved, abs(fd_free - ana) / (abs(ana) + 1e-3))
    assert worst <= 1e-7          # the analytic gradient treats s as a constant ...
    assert moved >= 1e-2          # ... and differs from the derivative of the un-frozen loss


# ---------------------------------------------------------------- invariants that hold at any size
def test_invariants():
    T, d, V, K = 64, 16, 50, 8
    H, W, y, valid = _rand_problem(10, T, d, V, masked=True)
    fwd, dH, dW = O.cat_forward_backward(H, W, y, valid, K, g=2.0)
    ok = fwd["eff_valid"]
    # sum_v dz[r, v] = 0  =>  dW summed over the vocabulary vanishes
    assert np.allclose(dW.sum(axis=0), 0, atol=1e-15)
    assert np.all(dH[~ok] == 0)
    p = np.exp(H @ W.T - fwd["lse"][:, None])
    assert np.allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-12)
    coef = 2.0 * fwd["weight"] / fwd["n_valid"]
    expect = coef[:, None] * (p @ W - W[np.where(ok, y, 0)])
    assert np.allclose(dH[ok], expect[ok], rtol=1e-10, atol=1e-16)
    rows = np.array([3, 17, 40])
    sub = dict(lse=fwd["lse"][rows], weight=fwd["weight"][rows], eff_valid=ok[rows])
    assert np.allclose(O.cat_dH_rows(H, W, y, sub, rows, fwd["n_valid"], g=2.0), dH[rows], rtol=1e-12, atol=1e-18)
    vs = np.array([0, 7, 49, int(y[0])])
    assert np.allclose(O.cat_dW_rows(H, W, y, fwd, vs, g=2.0), dW[vs], rtol=1e-12, atol=1e-18)


def test_all_invalid_gives_zero():
    H, W, y, _ = _rand_problem(11, 8, 4, 9)
    fwd, dH, dW = O.cat_forward_backward(H, W, y, np.zeros(8, np.uint8), 4)
    assert fwd["loss"] == 0.0 and fwd["n_valid"] == 0 and not dH.any() and not dW.any()


def test_row_chunking_does_not_change_results():
    H, W, y, valid = _rand_problem(12, 40, 8, 33, masked=True)
    a = O.cat_forward_backward(H, W, y, valid, 4, row_chunk=1024)
    b = O.cat_forward_backward(H, W, y, valid, 4, row_chunk=7)
    assert math.isclose(a[0]["loss"], b[0]["loss"], rel_tol=1e-14)
    assert np.allclose(a[1], b[1], rtol=1e-13, atol=1e-18) and np.allclose(a[2], b[2], rtol=1e-12, atol=1e-18)


# ---------------------------------------------------------------- binary32 weight routine
def test_weights_f32_is_sequential_binary32_with_denormals():
    rng = np.random.default_rng(13)
    K = 32
    c = rng.random(3 * K).astype(np.float32) * np.float32(0.2)
    ok = np.ones(3 * K, bool); ok[40] = False
    w = O.cat_weights_f32(c, ok, K)
    for b in range(3):
        s = np.float32(1.0)
        for k in range(K):
            r = b * K + k
            if ok[r]:
                assert w[r].tobytes() == s.tobytes()
                s = np.float32(s * c[r])
            else:
                assert w[r] == 0
    # V^-k underflows gradually: denormal results are kept, not flushed
    c = np.full(16, np.float32(2.0 ** -10), np.float32)
    w = O.cat_weights_f32(c, np.ones(16, bool), 16)
    assert w[14] == np.float32(2.0 ** -140) and w[14] != 0 and w[15] == 0


# ---------------------------------------------------------------- Eq. 12: CE + KD under the CAT weight
def _kd_problem(seed, B=5, K=4, d=8, dt=6, V=32, masked=False):
    rng = np.random.default_rng(seed)
    T, L = B * K, B + K - 1
    H, W = rng.standard_normal((T, d)), rng.standard_normal((V, d)) * 0.3
    Ht, Wt = rng.standard_normal((L, dt)), rng.standard_normal((V, dt)) * 0.5
    y = rng.integers(0, V, T)
    valid = np.ones(T, np.uint8)
    if masked:
        valid[rng.random(T) < 0.25] = 0
    return H, W, y, valid, Ht, Wt, np.arange(B)


def test_eq12_against_library_kl_and_cross_entropy_with_unit_weights():
    H, W, y, valid, Ht, Wt, st = _kd_problem(31, masked=True)
    K, beta = 4, 0.1
    fwd, dH, dW = O.cat_kd_forward_backward(H, W, y, valid, K, Ht, Wt, st, beta, conf_ext=np.ones(len(y)))
    t_row = O.kd_target_rows(st, K, len(y))
    ok = valid.astype(bool)
    Hg = torch.tensor(H, requires_grad=True)
    Wg = torch.tensor(W, requires_grad=True)
    logq = torch.log_softmax(Hg @ Wg.T, dim=1)
    p_t = torch.softmax(torch.tensor(Ht[t_row] @ Wt.T), dim=1)
    kd = torch.nn.functional.kl_div(logq, p_t, reduction="none").sum(dim=1)      # KL(p_t || q) per row
    ce = torch.nn.functional.nll_loss(logq, torch.tensor(y), reduction="none")
    m = torch.tensor(ok)
    loss = ((beta * ce + kd) * m).sum() / m.sum()
    loss.backward()
    assert math.isclose(fwd["loss"], loss.item(), rel_tol=1e-12)
    assert math.isclose(fwd["loss"], beta * fwd["loss_ce"] + fwd["loss_kd"], rel_tol=1e-14)
    assert np.allclose(dH, Hg.grad.numpy(), rtol=1e-10, atol=1e-15)
    assert np.allclose(dW, Wg.grad.numpy(), rtol=1e-10, atol=1e-15)
    assert np.all(fwd["row_kd"] >= -1e-15)


def test_eq12_special_targets():
    H, W, y, valid, Ht, Wt, st = _kd_problem(32)
    K, beta, T = 4, 0.1, len(y)
    cat, dH_c, dW_c = O.cat_forward_backward(H, W, y, valid, K, conf_ext=np.full(T, 0.5))
    # (a) a target that puts all its mass on the label: KL(onehot || q) = -log q_y = CE, so the loss is (1 + beta) CAT
    t_row = O.kd_target_rows(st, K, T)
    #     one target row serves several draft rows, so give every draft row its own position: block_start = b * K
    Ht_a = np.zeros((T, 32)); Wt_a = 60.0 * np.eye(32)
    Ht_a[np.arange(T), y] = 1.0
    fa, dH_a, dW_a = O.cat_kd_forward_backward(H, W, y, valid, K, Ht_a, Wt_a, np.arange(T // K) * K, beta, conf_ext=np.full(T, 0.5))
    assert math.isclose(fa["loss_kd"], cat["loss"], rel_tol=1e-12) and math.isclose(fa["loss"], (1 + beta) * cat["loss"], rel_tol=1e-12)
    assert np.allclose(dH_a, (1 + beta) * dH_c, rtol=1e-10, atol=1e-16) and np.allclose(dW_a, (1 + beta) * dW_c, rtol=1e-10, atol=1e-16)
    #     and with the target as confidence source (Eq. 9) a certain target gives unit weights
    fa2, _, _ = O.cat_kd_forward_backward(H, W, y, valid, K, Ht_a, Wt_a, np.arange(T // K) * K, beta, want_grads=False)
    assert np.allclose(fa2["weight"], 1.0, rtol=0, atol=1e-12)
    # (b) a target equal to the draft: KD = 0 with zero gradient, leaving beta * CAT
    fb, dH_b, dW_b = O.cat_kd_forward_backward(H, W, y, valid, K, H, W, np.arange(T // K) * K, beta, conf_ext=np.full(T, 0.5))
    assert abs(fb["loss_kd"]) <= 1e-15 and math.isclose(fb["loss"], beta * cat["loss"], rel_tol=1e-12)
    assert np.allclose(dH_b, beta * dH_c, rtol=1e-10, atol=1e-16) and np.allclose(dW_b, beta * dW_c, rtol=1e-10, atol=1e-16)
    # (c) uniform target against a uniform draft (W = 0): KD = 0; against a non-uniform draft: KD = mean(-log q) - log V
    fc, _, _ = O.cat_kd_forward_backward(H, np.zeros_like(W), y, valid, K, Ht, np.zeros_like(Wt), st, beta, conf_ext=np.ones(T), want_grads=False)
    assert abs(fc["loss_kd"]) <= 1e-15
    fd, _, _ = O.cat_kd_forward_backward(H, W, y, valid, K, Ht, np.zeros_like(Wt), st, beta, conf_ext=np.ones(T), want_grads=False)
    z = H @ W.T
    logq = z - np.log(np.exp(z).sum(axis=1, keepdims=True))
    assert math.isclose(fd["loss_kd"], float((-logq.mean(axis=1) - math.log(32)).mean()), rel_tol=1e-12)


def test_eq12_target_rows_are_shared_along_n_plus_k_and_weights_follow_eq9():
    H, W, y, valid, Ht, Wt, st = _kd_problem(33, B=6, K=4)
    K, T, L = 4, len(y), Ht.shape[0]
    fwd, _, _ = O.cat_kd_forward_backward(H, W, y, valid, K, Ht, Wt, st, 0.1, want_grads=False)
    t_row = fwd["target_row"].reshape(-1, K)
    assert t_row[1, 2] == t_row[2, 1] == t_row[3, 0] == 3                        # (n, k) -> n + k
    assert np.array_equal(fwd["lse_t"].reshape(-1, K)[1, 2], fwd["lse_t"].reshape(-1, K)[3, 0])
    # Eq. 9 as printed: the confidence is the target's probability of the row's label
    zt = Ht @ Wt.T
    p_t = np.exp(zt - np.log(np.exp(zt).sum(axis=1, keepdims=True)))
    expect_c = p_t[fwd["target_row"], y]
    assert np.allclose(fwd["conf"], expect_c, rtol=1e-13)
    assert np.array_equal(fwd["weight"], O.cat_weights(fwd["conf"], np.ones(T, bool), K))
    # a block whose positions run past the end of the sequence: those rows are invalid
    f2, dH2, _ = O.cat_kd_forward_backward(H, W, y, valid, K, Ht, Wt, st + 2, 0.1)
    bad = (O.kd_target_rows(st + 2, K, T) >= L)
    assert bad.any() and not f2["eff_valid"][bad].any() and f2["eff_valid"][~bad].all()
    assert not dH2[bad].any() and f2["n_valid"] == int((~bad).sum())


def test_eq12_gradients_match_finite_differences_with_frozen_weights():
    H, W, y, valid, Ht, Wt, st = _kd_problem(34, B=3, K=4, masked=True)
    K, beta, g = 4, 0.1, 0.7
    fwd, dH, dW = O.cat_kd_forward_backward(H, W, y, valid, K, Ht, Wt, st, beta, g=g)
    w, N = fwd["weight"], fwd["n_valid"]

    def frozen(Hx, Wx):
        f, _, _ = O.cat_kd_forward_backward(Hx, Wx, y, valid, K, Ht, Wt, st, beta, conf_ext=np.ones(len(y)), want_grads=False)
        return g * float((w * (beta * f["row_ce"] + f["row_kd"])).sum() / N)

    eps = 1e-6
    rng = np.random.default_rng(0)
    for _ in range(12):
        r, i = rng.integers(0, H.shape[0]), rng.integers(0, H.shape[1])
        Hp, Hm = H.copy(), H.copy(); Hp[r, i] += eps; Hm[r, i] -= eps
        assert math.isclose((frozen(Hp, W) - frozen(Hm, W)) / (2 * eps), dH[r, i], rel_tol=1e-6, abs_tol=1e-10)
        v, j = rng.integers(0, W.shape[0]), rng.integers(0, W.shape[1])
        Wp, Wm = W.copy(), W.copy(); Wp[v, j] += eps; Wm[v, j] -= eps
        assert math.isclose((frozen(H, Wp) - frozen(H, Wm)) / (2 * eps), dW[v, j], rel_tol=1e-6, abs_tol=1e-10)
    # each row of dz sums to zero (both softmaxes and the one-hot have unit mass): columns of dW summed over v vanish
    assert np.allclose(dW.sum(axis=0), 0.0, atol=1e-14)


@pytest.mark.parametrize("source", ["target", "draft"])
def test_eq12_sampled_block_routine_agrees_with_the_whole_batch_routine(source):
    H, W, y, valid, Ht, Wt, st = _kd_problem(35, B=9, K=4, masked=True)
    fwd, dH, _ = O.cat_kd_forward_backward(H, W, y, valid, 4, Ht, Wt, st, 0.1, conf_source=source, g=0.5, row_chunk=7)
    rows, out, dH_rows = O.cat_kd_rows(H, W, y, valid, 4, Ht, Wt, st, 0.1, [0, 3, 8], fwd["n_valid"], conf_source=source, g=0.5)
    assert np.array_equal(rows, np.r_[0:4, 12:16, 32:36])
    for key in ("lse", "lse_t", "conf", "weight", "row_ce", "row_kd"):
        assert np.allclose(out[key], fwd[key][rows], rtol=1e-13, atol=0), key
    assert np.allclose(dH_rows, dH[rows], rtol=1e-12, atol=1e-18)


def test_eq12_draft_confidence_source_is_the_heads_own_confidence():
    # conf_source="draft": the Eq. 9 confidences are the draft head's own label probabilities, i.e. those of the
    # plain CAT forward pass (pinned above against a library softmax), and the weights their Eq. 10 products
    H, W, y, valid, Ht, Wt, st = _kd_problem(36, B=7, K=4, masked=True)
    fwd, _, _ = O.cat_kd_forward_backward(H, W, y, valid, 4, Ht, Wt, st, 0.1, conf_source="draft", want_grads=False)
    ok = fwd["eff_valid"]
    plain = O.cat_forward(H, W, y, ok.astype(np.uint8), 4)
    assert np.array_equal(plain["eff_valid"], ok)
    assert np.allclose(fwd["conf"], plain["conf"], rtol=1e-13, atol=0)
    assert np.allclose(fwd["weight"], plain["weight"], rtol=1e-12, atol=0)
    tgt, _, _ = O.cat_kd_forward_backward(H, W, y, valid, 4, Ht, Wt, st, 0.1, conf_source="target", want_grads=False)
    assert not np.allclose(tgt["conf"][ok], fwd["conf"][ok])

"""fp64 CPU oracle for the Confidence-Adaptive Token (CAT) loss and its gradients.

THIS IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, obviously
correct restatement of what the paper's training objective computes, written
from the formulas (PARD-2, Section 3.2 "Confidence-Adaptive Token Optimization
Strategy", Eq. 9, Eq. 10, Eq. 11, and Section 3.3 Eq. 12).  Only the tests, the
smoke check and the benchmark's CPU-baseline leg may import it.  It shares no
code with the CUDA path and never imports it.

Everything is numpy float64.  The only library primitive used as a step is the
matrix product for the logits (and for the two gradient contractions); rows are
processed in chunks purely to bound memory -- rows are independent, so chunking
changes nothing but the order in which dW's sum over rows is accumulated.

Notation (Section 3.2): a draft block has K parallel positions k = 0..K-1; the
rows of H are laid out block after block, row r = b*K + k.  y_r is the
ground-truth token of row r.  c_k is the confidence in y at position k (Eq. 9),
s_k the exclusive prefix product of confidences (Eq. 10), used as a
stop-gradient weight on the per-token cross-entropy (Eq. 11).

Readings taken where the paper is silent (each also listed in the design notes):
  * confidence source: the paper's Eq. 9 uses the target model's probability of
    the label.  Here the default is the probability the head itself (H, W)
    assigns to the label; `conf_ext` supplies externally computed confidences
    (the paper's target-model mode).  Either way the weight is a constant under
    differentiation (sentence after Eq. 10: "stop-gradient weight").
  * normalisation: Eq. 11 has 1/K for one block; over a batch with a valid-row
    mask the loss is divided by N = number of valid rows (equals the mean over
    blocks of Eq. 11 when all rows are valid; equals mean CE for unit weights,
    Eq. 5).
  * invalid rows (padding, rows past the sequence end in Eq. 12's n <= N-k):
    weight 0, no loss, no gradient, and factor 1 in the prefix product.
  * a label outside [0, V) on a valid row makes the row invalid.

Beside the CAT objective: the fixed position decay gamma**k that the paper ablates CAT
against (Table 3), the per-block acceptance-length estimate of Eq. 8, and the target-model
confidences of Eq. 9 laid out as draft rows (Eq. 12's s_{n,k}).

Pins (tests/test_oracle_pins.py): Eq. 5 degenerate case against
torch.nn.functional.cross_entropy, K = 1, constant confidence = fixed decay
gamma**k, W = 0 closed form, the Eq. 6/Eq. 8 acceptance-length identity, a hand
example, finite differences with frozen weights, brute force in pure Python.
Parity unpinned by the paper (fixed by the readings above): the confidence
source, the batch normaliser, and the treatment of masked rows.
"""
from __future__ import annotations

import numpy as np

__all__ = [
    "effective_valid",
    "softmax_stats",
    "cat_weights",
    "cat_weights_f32",
    "fixed_decay_weights",
    "fixed_decay_weights_f32",
    "accept_len_estimate",
    "target_confidence",
    "window_confidence",
    "cat_forward",
    "cat_forward_from_row_stats",
    "cat_backward",
    "cat_forward_backward",
    "cat_dH_rows",
    "cat_dW_rows",
    "kd_target_rows",
    "cat_kd_forward_backward",
    "cat_kd_rows",
]


def _as_f64(x) -> np.ndarray:
    """Widen an array-like (numpy, or a torch CPU tensor incl. bf16) to float64 exactly."""
    if hasattr(x, "detach"):  # torch tensor, without importing torch here
        x = x.detach().to("cpu").double().numpy()
    return np.ascontiguousarray(x, dtype=np.float64)


def _as_i64(x) -> np.ndarray:
    if hasattr(x, "detach"):
        x = x.detach().to("cpu").numpy()
    return np.ascontiguousarray(x, dtype=np.int64)


def effective_valid(labels, valid, V: int) -> np.ndarray:
    """Row r takes part iff its mask bit is set and 0 <= y_r < V (boolean array)."""
    y = _as_i64(labels)
    ok = (y >= 0) & (y < V)
    if valid is not None:
        v = valid.detach().to("cpu").numpy() if hasattr(valid, "detach") else np.asarray(valid)
        ok &= v.astype(bool)
    return ok


def softmax_stats(z: np.ndarray):
    """Row-wise m = max z, l = sum exp(z - m), lse = m + log l (the log-partition in Eq. 11's log P)."""
    m = z.max(axis=1)
    l = np.exp(z - m[:, None]).sum(axis=1)
    return m, l, m + np.log(l)


def cat_weights(conf: np.ndarray, eff_valid: np.ndarray, K: int) -> np.ndarray:
    """Eq. 10: s_k = prod_{j<k} c_j, s_0 = 1, independently inside every block of K rows.

    Invalid rows get weight 0 and contribute the factor 1 to the product.
    Sequential in k (left to right), float64.
    """
    c = np.asarray(conf, dtype=np.float64).reshape(-1, K)
    ok = np.asarray(eff_valid, dtype=bool).reshape(-1, K)
    w = np.zeros_like(c)
    s = np.ones(c.shape[0], dtype=np.float64)
    for k in range(K):
        w[:, k] = np.where(ok[:, k], s, 0.0)
        s = np.where(ok[:, k], s * c[:, k], s)
    return w.reshape(-1)


def cat_weights_f32(conf_f32: np.ndarray, eff_valid: np.ndarray, K: int) -> np.ndarray:
    """Eq. 10 in IEEE binary32, left to right, round-to-nearest-even, denormals kept.

    Reference for the bit-exact weight check: given float32 confidences it
    returns the float32 sequential product ((1*c_0)*c_1)*... per block.
    """
    c = np.asarray(conf_f32)
    if c.dtype != np.float32:
        raise TypeError("cat_weights_f32 wants float32 confidences")
    c = c.reshape(-1, K)
    ok = np.asarray(eff_valid, dtype=bool).reshape(-1, K)
    w = np.zeros_like(c)
    s = np.ones(c.shape[0], dtype=np.float32)
    for k in range(K):
        w[:, k] = np.where(ok[:, k], s, np.float32(0.0))
        s = np.where(ok[:, k], (s * c[:, k]).astype(np.float32), s)
    return w.reshape(-1)


def fixed_decay_weights(gamma: float, eff_valid: np.ndarray, K: int) -> np.ndarray:
    """The fixed position decay the paper ablates CAT against (Section 4.3, Table 3):
    the weight of draft position k is gamma**k whatever the confidences are; k counts
    positions, so masked rows in between still advance the exponent.  Invalid rows get 0.
    Sequential product (1*gamma)*gamma*..., float64."""
    ok = np.asarray(eff_valid, dtype=bool).reshape(-1, K)
    w = np.zeros(ok.shape, dtype=np.float64)
    s = 1.0
    for k in range(K):
        w[:, k] = np.where(ok[:, k], s, 0.0)
        s = s * float(gamma)
    return w.reshape(-1)


def fixed_decay_weights_f32(gamma, eff_valid: np.ndarray, K: int) -> np.ndarray:
    """fixed_decay_weights in IEEE binary32: ((1*g)*g)*... with g = float32(gamma)."""
    ok = np.asarray(eff_valid, dtype=bool).reshape(-1, K)
    g = np.float32(gamma)
    w = np.zeros(ok.shape, dtype=np.float32)
    s = np.float32(1.0)
    for k in range(K):
        w[:, k] = np.where(ok[:, k], s, np.float32(0.0))
        s = np.float32(s * g)
    return w.reshape(-1)


def accept_len_estimate(conf: np.ndarray, weight: np.ndarray, K: int) -> np.ndarray:
    """Per-block estimate of the expected acceptance length, Eq. 8 with the estimates of
    Eq. 9 and Eq. 10 in place of a_k and s_k:  sum_k s_k * c_k  (invalid rows have s_k = 0)."""
    c = np.asarray(conf, dtype=np.float64).reshape(-1, K)
    w = np.asarray(weight, dtype=np.float64).reshape(-1, K)
    return (w * c).sum(axis=1)


def target_confidence(Ht, Wt, labels, valid=None, row_chunk: int = 1024):
    """Eq. 9: the probability the TARGET model gives the ground-truth token of every sequence
    position, teacher-forced: c_i = softmax(Ht[i] . Wt^T)[y_i].  Ht [L, d_t] are the target's
    final hidden states, Wt [V, d_t] its LM head.  Returns (conf[L], lse[L]); positions that
    are masked or whose label is outside [0, V) get confidence 1."""
    Hd, Wd, y = _as_f64(Ht), _as_f64(Wt), _as_i64(labels)
    L = Hd.shape[0]
    ok = effective_valid(y, valid, Wd.shape[0])
    ysafe = np.where(ok, y, 0)
    lse = np.empty(L)
    zy = np.empty(L)
    for r0 in range(0, L, row_chunk):
        r1 = min(L, r0 + row_chunk)
        z = Hd[r0:r1] @ Wd.T
        _, _, lse[r0:r1] = softmax_stats(z)
        zy[r0:r1] = z[np.arange(r1 - r0), ysafe[r0:r1]]
    return np.where(ok, np.exp(zy - lse), 1.0), lse


def window_confidence(conf_seq: np.ndarray, block_start, K: int) -> np.ndarray:
    """Lay per-position target confidences out as draft rows (Eq. 12's s_{n,k}): the block that
    drafts positions start..start+K-1 of the flattened sequence gets conf_ext[b*K + k] =
    conf_seq[start_b + k]; positions outside [0, L) get 1 (those rows are invalid anyway).
    Eq. 10 applied to these rows is the sliding-window product over the sequence."""
    c = np.asarray(conf_seq, dtype=np.float64)
    st = _as_i64(block_start)
    L = c.shape[0]
    out = np.ones((st.shape[0], K), dtype=np.float64)
    for b in range(st.shape[0]):
        for k in range(K):
            i = int(st[b]) + k
            if 0 <= i < L:
                out[b, k] = c[i]
    return out.reshape(-1)


def cat_forward(H, W, labels, valid, K: int, conf_ext=None, row_chunk: int = 1024,
                check_rows_sum_to_one: bool = True, fixed_decay_gamma=None) -> dict:
    """Forward pass of the CAT objective (Eq. 9-11) over T = B*K rows.

    Returns a dict with float64 arrays lse[T], z_label[T], conf[T], weight[T],
    row_ce[T] (= -log P(y_r), 0 on invalid rows), eff_valid[T] (bool),
    n_valid (int) and the scalar loss = (1/N) sum_r w_r * row_ce_r.
    """
    Hd, Wd, y = _as_f64(H), _as_f64(W), _as_i64(labels)
    T, d = Hd.shape
    V = Wd.shape[0]
    if Wd.shape[1] != d or y.shape[0] != T or K < 1 or T % K != 0:
        raise ValueError("bad shapes")
    ok = effective_valid(y, valid, V)
    ysafe = np.where(ok, y, 0)
    lse = np.empty(T)
    zy = np.empty(T)
    for r0 in range(0, T, row_chunk):
        r1 = min(T, r0 + row_chunk)
        z = Hd[r0:r1] @ Wd.T                       # logits of these rows over the whole vocabulary
        _, _, lse[r0:r1] = softmax_stats(z)
        if check_rows_sum_to_one:
            p_sum = np.exp(z - lse[r0:r1, None]).sum(axis=1)
            assert np.all(np.abs(p_sum - 1.0) <= 1e-12), "softmax rows do not sum to 1"
        zy[r0:r1] = z[np.arange(r1 - r0), ysafe[r0:r1]]
    return cat_forward_from_row_stats(lse, zy, y, valid, K, V, conf_ext=conf_ext, fixed_decay_gamma=fixed_decay_gamma)


def cat_forward_from_row_stats(lse, z_label, labels, valid, K: int, V: int, conf_ext=None, fixed_decay_gamma=None) -> dict:
    """Eq. 9-11 once the per-row log-partition lse[T] and label logit z_label[T] are known (the
    second half of cat_forward; also used to rebuild a forward state from stored lse / z_label)."""
    lse, zy, y = np.asarray(lse, dtype=np.float64), np.asarray(z_label, dtype=np.float64), _as_i64(labels)
    ok = effective_valid(y, valid, V)
    p_label = np.exp(zy - lse)                      # probability of the label token
    if conf_ext is None:
        conf = np.where(ok, p_label, 1.0)           # Eq. 9 evaluated with this head
    else:
        conf = np.where(ok, _as_f64(conf_ext), 1.0)  # Eq. 9 from the target model, supplied
    if fixed_decay_gamma is None:
        w = cat_weights(conf, ok, K)                # Eq. 10
    else:
        w = fixed_decay_weights(fixed_decay_gamma, ok, K)   # the ablation baseline: gamma**k
    row_ce = np.where(ok, lse - zy, 0.0)            # -log P(y_r)
    n_valid = int(ok.sum())
    loss = float((w * row_ce).sum() / n_valid) if n_valid > 0 else 0.0   # Eq. 11, batch mean
    return dict(loss=loss, lse=lse, z_label=zy, conf=conf, weight=w, row_ce=row_ce,
                eff_valid=ok, n_valid=n_valid)


def cat_backward(H, W, labels, K: int, fwd: dict, g: float = 1.0, row_chunk: int = 1024):
    """Gradients of g * loss w.r.t. H and W with the weights held constant (stop-gradient).

    dz[r, v] = g * (w_r / N) * (p[r, v] - [v == y_r]);  dH = dz W;  dW = dz^T H.
    """
    Hd, Wd, y = _as_f64(H), _as_f64(W), _as_i64(labels)
    T, d = Hd.shape
    V = Wd.shape[0]
    ok, w, lse, N = fwd["eff_valid"], fwd["weight"], fwd["lse"], fwd["n_valid"]
    dH = np.zeros((T, d))
    dW = np.zeros((V, d))
    if N == 0:
        return dH, dW
    coef = np.where(ok, g * w / N, 0.0)
    ysafe = np.where(ok, y, 0)
    for r0 in range(0, T, row_chunk):
        r1 = min(T, r0 + row_chunk)
        z = Hd[r0:r1] @ Wd.T
        p = np.exp(z - lse[r0:r1, None])
        p[np.arange(r1 - r0), ysafe[r0:r1]] -= 1.0
        dz = p * coef[r0:r1, None]
        dH[r0:r1] = dz @ Wd
        dW += dz.T @ Hd[r0:r1]
    return dH, dW


def cat_forward_backward(H, W, labels, valid, K: int, conf_ext=None, g: float = 1.0,
                         row_chunk: int = 1024, fixed_decay_gamma=None):
    fwd = cat_forward(H, W, labels, valid, K, conf_ext=conf_ext, row_chunk=row_chunk,
                      fixed_decay_gamma=fixed_decay_gamma)
    dH, dW = cat_backward(H, W, labels, K, fwd, g=g, row_chunk=row_chunk)
    return fwd, dH, dW


def cat_dH_rows(H, W, labels, fwd_rows: dict, rows: np.ndarray, n_valid_total: int, g: float = 1.0):
    """dH for a chosen set of rows, given the forward state of exactly those rows.

    `fwd_rows` holds lse / weight / eff_valid for `rows` (in that order);
    `n_valid_total` is N of the whole batch.
    """
    Hd, Wd, y = _as_f64(H), _as_f64(W), _as_i64(labels)
    rows = np.asarray(rows, dtype=np.int64)
    ok = fwd_rows["eff_valid"]
    z = Hd[rows] @ Wd.T
    p = np.exp(z - fwd_rows["lse"][:, None])
    p[np.arange(len(rows)), np.where(ok, y[rows], 0)] -= 1.0
    coef = np.where(ok, g * fwd_rows["weight"] / n_valid_total, 0.0)
    return (p * coef[:, None]) @ Wd


def cat_dW_rows(H, W, labels, fwd: dict, vocab_rows: np.ndarray, g: float = 1.0):
    """dW[v, :] for chosen token ids v, given the forward state of ALL rows."""
    Hd, Wd, y = _as_f64(H), _as_f64(W), _as_i64(labels)
    v = np.asarray(vocab_rows, dtype=np.int64)
    ok, N = fwd["eff_valid"], fwd["n_valid"]
    z = Hd @ Wd[v].T                                  # [T, len(v)]
    p = np.exp(z - fwd["lse"][:, None])
    p -= (y[:, None] == v[None, :]) & ok[:, None]
    coef = np.where(ok, g * fwd["weight"] / N, 0.0)
    return (p * coef[:, None]).T @ Hd


# ------------------------------------------------------------------------------------------
# Section 3.3, Eq. 12: the full PARD-2 training loss, cross-entropy plus distillation from
# the target model, both under the same prefix-indexed weight s_{n,k}.
#
# Readings (the paper names the distillation loss without writing it out):
#   * L^KD of a row is the forward KL divergence from the target's next-token distribution
#     p^t to the draft's q, both plain softmaxes (temperature 1) over the shared vocabulary:
#         L^KD = sum_v p^t_v (log p^t_v - log q_v).
#     Its gradient w.r.t. the draft logits is q - p^t; the target side receives no gradient.
#   * The target distribution of draft row (n, k) is the target's teacher-forced distribution at
#     sequence position n + k: it depends on the absolute position only, so one target row
#     serves every draft row that predicts that position.  Draft row (b, k) uses target row
#     block_start[b] + k of Ht; a row whose target position falls outside [0, L) is invalid.
#   * Batch normaliser as for Eq. 11: divide by N = number of valid rows.
#   * The weights may come from the target's confidence in the label (Eq. 9 as printed:
#     c = p^t[y]), from the draft's own (the default of the plain CAT entry points), or from
#     the caller (conf_ext).  They are constants under differentiation either way.
# ------------------------------------------------------------------------------------------
def kd_target_rows(block_start, K: int, T: int) -> np.ndarray:
    """Target row of every draft row: t[b*K + k] = block_start[b] + k."""
    st = _as_i64(block_start)
    if st.shape[0] * K != T:
        raise ValueError("block_start must have T / K entries")
    return (st[:, None] + np.arange(K)[None, :]).reshape(-1)


def _kd_row_stats(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows):
    """Per-row pieces of Eq. 12 for the given draft rows: log-partitions of both sides,
    CE = -log q_y, KD = sum_v p_v (log p_v - log q_v), and the label probabilities q_y, p_y."""
    z = Hd[rows] @ Wd.T                              # draft logits
    zt = Htd[tsafe[rows]] @ Wtd.T                    # target logits of each row's sequence position
    _, _, lse = softmax_stats(z)
    _, _, lse_t = softmax_stats(zt)
    logq = z - lse[:, None]
    logp = zt - lse_t[:, None]
    p_t = np.exp(logp)
    i = np.arange(len(rows))
    yy = ysafe[rows]
    return dict(lse=lse, lse_t=lse_t, ce=-logq[i, yy], kd=(p_t * (logp - logq)).sum(axis=1),
                q_y=np.exp(logq[i, yy]), p_y=p_t[i, yy], q=np.exp(logq), p_t=p_t)


def cat_kd_forward_backward(H, W, labels, valid, K: int, Ht, Wt, block_start, beta: float,
                            conf_source: str = "target", conf_ext=None, g: float = 1.0,
                            fixed_decay_gamma=None, want_grads: bool = True, row_chunk: int = 512):
    """loss = (1/N) sum_r s_r (beta * CE_r + KD_r)  (Eq. 12 summed over k and n), its parts, and
    the gradients of g * loss w.r.t. H and W with s held constant.

    Returns (fwd dict, dH, dW).  fwd has loss, loss_ce, loss_kd (each already divided by N, so
    loss = beta*loss_ce + loss_kd), lse, lse_t (per draft row), conf, weight, row_ce, row_kd,
    eff_valid, n_valid, target_row.  Rows are processed in chunks only to bound memory.
    """
    Hd, Wd, y = _as_f64(H), _as_f64(W), _as_i64(labels)
    Htd, Wtd = _as_f64(Ht), _as_f64(Wt)
    T, d = Hd.shape
    V = Wd.shape[0]
    L = Htd.shape[0]
    if Wtd.shape[0] != V or Wtd.shape[1] != Htd.shape[1] or T % K != 0:
        raise ValueError("bad shapes")
    t_row = kd_target_rows(block_start, K, T)
    ok = effective_valid(y, valid, V) & (t_row >= 0) & (t_row < L)
    ysafe = np.where(ok, y, 0)
    tsafe = np.where(ok, t_row, 0)
    lse, lse_t, ce, kdv, q_y, p_y = (np.empty(T) for _ in range(6))
    for r0 in range(0, T, row_chunk):
        rows = np.arange(r0, min(T, r0 + row_chunk))
        st = _kd_row_stats(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows)
        lse[rows], lse_t[rows], ce[rows], kdv[rows], q_y[rows], p_y[rows] = st["lse"], st["lse_t"], st["ce"], st["kd"], st["q_y"], st["p_y"]
    row_ce = np.where(ok, ce, 0.0)                                       # L^CE
    row_kd = np.where(ok, kdv, 0.0)                                      # L^KD = KL(p^t || q)
    if conf_ext is not None:
        conf = np.where(ok, _as_f64(conf_ext), 1.0)
    elif conf_source == "target":
        conf = np.where(ok, p_y, 1.0)                                    # Eq. 9 as printed
    elif conf_source == "draft":
        conf = np.where(ok, q_y, 1.0)
    else:
        raise ValueError("conf_source must be 'target' or 'draft'")
    w = cat_weights(conf, ok, K) if fixed_decay_gamma is None else fixed_decay_weights(fixed_decay_gamma, ok, K)
    N = int(ok.sum())
    loss_ce = float((w * row_ce).sum() / N) if N else 0.0
    loss_kd = float((w * row_kd).sum() / N) if N else 0.0
    fwd = dict(loss=beta * loss_ce + loss_kd, loss_ce=loss_ce, loss_kd=loss_kd, lse=lse, lse_t=lse_t, conf=conf,
               weight=w, row_ce=row_ce, row_kd=row_kd, eff_valid=ok, n_valid=N, target_row=t_row)
    if not want_grads:
        return fwd, None, None
    dH = np.zeros((T, d))
    dW = np.zeros((V, d))
    if N:
        coef = np.where(ok, g * w / N, 0.0)
        for r0 in range(0, T, row_chunk):
            rows = np.arange(r0, min(T, r0 + row_chunk))
            dz = _kd_dz(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows, coef, beta)
            dH[rows] = dz @ Wd
            dW += dz.T @ Hd[rows]
    return fwd, dH, dW


def _kd_dz(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows, coef, beta):
    """dz of Eq. 12 for the given rows: coef_r * (beta (q - onehot) + (q - p_t))."""
    st = _kd_row_stats(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows)
    onehot = np.zeros_like(st["q"])
    onehot[np.arange(len(rows)), ysafe[rows]] = 1.0
    return coef[rows, None] * (beta * (st["q"] - onehot) + (st["q"] - st["p_t"]))


def cat_kd_rows(H, W, labels, valid, K: int, Ht, Wt, block_start, beta: float, blocks, n_valid_total: int,
                conf_source: str = "target", g: float = 1.0):
    """Eq. 12 for a chosen set of whole draft blocks of a large batch (sampled full-size checks):
    per-row lse, lse_t, conf, weight, CE, KD of those blocks' rows, and their dH rows, given N of
    the whole batch.  Returns (rows, dict, dH_rows)."""
    Hd, Wd, y = _as_f64(H), _as_f64(W), _as_i64(labels)
    Htd, Wtd = _as_f64(Ht), _as_f64(Wt)
    T, V, L = Hd.shape[0], Wd.shape[0], Htd.shape[0]
    blocks = np.asarray(blocks, dtype=np.int64)
    rows = (blocks[:, None] * K + np.arange(K)[None, :]).reshape(-1)
    t_row = kd_target_rows(block_start, K, T)
    ok_all = effective_valid(y, valid, V) & (t_row >= 0) & (t_row < L)
    ysafe, tsafe = np.where(ok_all, y, 0), np.where(ok_all, t_row, 0)
    st = _kd_row_stats(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows)
    ok = ok_all[rows]
    conf = np.where(ok, st["p_y"] if conf_source == "target" else st["q_y"], 1.0)
    w = cat_weights(conf, ok, K)
    coef = np.zeros(T)
    coef[rows] = np.where(ok, g * w / n_valid_total, 0.0)
    dz = _kd_dz(Hd, Wd, Htd, Wtd, ysafe, tsafe, rows, coef, beta)
    out = dict(lse=st["lse"], lse_t=st["lse_t"], conf=conf, weight=w, row_ce=np.where(ok, st["ce"], 0.0),
               row_kd=np.where(ok, st["kd"], 0.0), eff_valid=ok)
    return rows, out, dz @ Wd

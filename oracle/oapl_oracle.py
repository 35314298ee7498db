"""fp64 CPU oracle for the OAPL LM-head hot path.  TEST INFRASTRUCTURE ONLY.

This module is the plain, slow, obviously-correct statement of what the CUDA
library computes.  It is imported only by the tests, by the smoke check and by
the benchmark's CPU-baseline leg; the product path never calls it and shares no
code with it.  Everything is float64 numpy; the only library primitive used as
a step is the dense matrix product.

What it states (OAPL paper, "Method" section):

* token log-probability  ln pi(y_t | x, y_<t) = z[y_t] - ln sum_v exp z[v] with
  z = h . W^T  (the policy's next-token distribution; the sequence quantity
  pi(y|x) of Eq. 3 is the product over the response tokens, so its log is the
  masked sum of the token log-probabilities);
* the group value estimate of Eq. 2, V^(x) = beta ln (1/G) sum_i exp(r_i/beta);
* the optimal-advantage estimate A_i = r_i - V^(x) (text below Eq. 2);
* the squared-regression objective of Eq. 3 with the two temperatures of the
  "Experimental Setup" section (beta_v in Eq. 2, beta_loss in Eq. 3);
* its gradient with respect to the hidden states H and the LM-head weight W,
  obtained by differentiating Eq. 3 through the softmax (Algorithm 1 performs
  gradient descent on Eq. 3; no gradient flows through V^ or through the
  inference engine's log-probabilities, which are data).

Pins (tests/test_oracle_pins.py): brute-force logits by explicit loops, softmax
normalisation, the W=0 and V=2 closed forms, scipy's logsumexp, the beta->0 and
beta->inf limits of Eq. 2, its binary-reward closed form and a 60-digit decimal
evaluation of the literal formula, zero loss and zero gradient at the
closed-form optimum, central finite differences of the loss, and the zero
column sum of dW; for the entropy statistic the literal -sum p ln p, the uniform
and two-token closed forms, scipy.stats.entropy and the bound 0 <= H <= ln V.  The paper prints no worked numeric example, so the numeric
end-to-end value of a whole step is "parity unpinned" beyond those pins.
"""
from __future__ import annotations

import numpy as np


# --------------------------------------------------------------------------
# input decoding
# --------------------------------------------------------------------------
def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Widen bfloat16 bit patterns (uint16) to float64 exactly.

    A bfloat16 is the upper half of an IEEE float32, so placing the 16 bits in
    the high half of a 32-bit word and reading it as float32 is exact, and
    float32 -> float64 is exact.
    """
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    as_f32 = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return as_f32.astype(np.float64)


# --------------------------------------------------------------------------
# token and sequence log-probabilities
# --------------------------------------------------------------------------
def logits(H: np.ndarray, W: np.ndarray) -> np.ndarray:
    """z[n, v] = sum_k H[n, k] * W[v, k]   (LM head without bias)."""
    return np.asarray(H, dtype=np.float64) @ np.asarray(W, dtype=np.float64).T


def log_sum_exp(z: np.ndarray) -> np.ndarray:
    """Row-wise natural-log ln sum_v exp z[n, v], shifted by the row maximum."""
    M = z.max(axis=1)
    return M + np.log(np.exp(z - M[:, None]).sum(axis=1))


def token_logprobs(H, W, targets, mask):
    """Per-row ln pi(target | prefix) and the row's log-sum-exp.

    H [N, d], W [V, d] float64; targets [N] int; mask [N] in {0,1}.
    Rows with mask == 0 give lp = 0 and lse = 0 and their target is ignored.
    Returns (lp [N], lse [N]).
    """
    H = np.asarray(H, dtype=np.float64)
    N = H.shape[0]
    mask = np.asarray(mask).astype(bool)
    targets = np.asarray(targets).astype(np.int64)
    lp = np.zeros(N)
    lse = np.zeros(N)
    live = np.flatnonzero(mask)
    if live.size:
        z = logits(H[live], W)
        l = log_sum_exp(z)
        lse[live] = l
        lp[live] = z[np.arange(live.size), targets[live]] - l
    return lp, lse


def sequence_sums(lp, logp_inf, mask, seq_id, S):
    """Masked per-sequence sums.

    s_i = sum_{n in seq i} m_n lp_n                (= ln pi(y_i | x), Eq. 3)
    D_i = sum_{n in seq i} m_n (lp_n - logp_inf_n) (= ln pi/pi_vllm, Eq. 3)
    T_i = sum_{n in seq i} m_n                     (response length)
    """
    m = np.asarray(mask).astype(np.float64)
    seq_id = np.asarray(seq_id).astype(np.int64)
    lp = np.asarray(lp, dtype=np.float64)
    q = np.asarray(logp_inf, dtype=np.float64)
    s = np.zeros(S)
    D = np.zeros(S)
    T = np.zeros(S)
    # where(mask) keeps unread logp_inf entries (possibly NaN) out of the sums
    diff = np.where(m > 0, lp - np.where(m > 0, q, 0.0), 0.0)
    np.add.at(s, seq_id, m * lp)
    np.add.at(D, seq_id, diff)
    np.add.at(T, seq_id, m)
    return s, D, T


# --------------------------------------------------------------------------
# Eq. 2: value estimate
# --------------------------------------------------------------------------
def value_estimate(reward, group_id, P, beta_v):
    """V^_p = beta ln( (1/G_p) sum_{i in group p} exp(r_i / beta) )   (Eq. 2).

    Evaluated in the algebraically identical max-shifted form so that small
    beta does not overflow.  G_p is the actual member count; a group without
    members gets 0.
    """
    r = np.asarray(reward, dtype=np.float64)
    g = np.asarray(group_id).astype(np.int64)
    vhat = np.zeros(P)
    for p in range(P):
        rp = r[g == p]
        if rp.size == 0:
            continue
        R = rp.max()
        vhat[p] = R + beta_v * np.log(np.mean(np.exp((rp - R) / beta_v)))
    return vhat


# --------------------------------------------------------------------------
# Eq. 3: loss
# --------------------------------------------------------------------------
def loss_from_sums(D, reward, group_id, P, beta_v, beta_loss, loss_scale):
    """Advantage, residual, loss and dL/ds_i from the per-sequence log-ratios.

    A_i     = r_i - V^_{g(i)}                    (text below Eq. 2)
    delta_i = beta_loss * D_i - A_i              (the bracket of Eq. 3)
    L       = loss_scale * sum_i delta_i^2       (Eq. 3; loss_scale = 1 is the
                                                  paper's plain double sum)
    c_i     = dL/dD_i = 2 loss_scale beta_loss delta_i
    """
    r = np.asarray(reward, dtype=np.float64)
    g = np.asarray(group_id).astype(np.int64)
    vhat = value_estimate(r, g, P, beta_v)
    A = r - vhat[g]
    delta = beta_loss * np.asarray(D, dtype=np.float64) - A
    loss = loss_scale * np.sum(delta * delta)
    coef = 2.0 * loss_scale * beta_loss * delta
    return dict(loss=loss, vhat=vhat, A=A, delta=delta, coef=coef)


def batch_stats(D, T, reward, group_id, vhat, P):
    """Diagnostics of one batch from the quantities of Eq. 2 / Eq. 3 (the paper tracks training
    curves; these are the scalars a trainer would log next to the loss):

      live_tokens            sum_i T_i
      mean_abs_log_ratio     mean over the sequences with T_i > 0 of |D_i|,  D_i = ln pi/pi_vllm (y_i|x)
      max_abs_log_ratio      max over the same sequences of |D_i|
      mean_token_log_ratio   sum_i D_i / sum_i T_i
      mean_advantage         mean over all sequences of A_i = r_i - V^_{g(i)}  (text below Eq. 2)
      frac_groups_all_equal  fraction of the groups with members whose rewards are all equal
                             (there A_i = 0: the term of Eq. 3 only pulls the log-ratio to 0)
      mean_reward            mean over all sequences of r_i
    Empty denominators give 0.
    """
    D = np.asarray(D, dtype=np.float64)
    T = np.asarray(T, dtype=np.float64)
    r = np.asarray(reward, dtype=np.float64)
    g = np.asarray(group_id).astype(np.int64)
    vhat = np.asarray(vhat, dtype=np.float64)
    live = T > 0
    n_live = T.sum()
    groups = [r[g == p] for p in range(P)]
    with_members = [x for x in groups if x.size]
    return dict(
        live_tokens=float(n_live),
        mean_abs_log_ratio=float(np.abs(D[live]).mean()) if live.any() else 0.0,
        max_abs_log_ratio=float(np.abs(D[live]).max()) if live.any() else 0.0,
        mean_token_log_ratio=float(D[live].sum() / n_live) if n_live > 0 else 0.0,
        mean_advantage=float((r - vhat[g]).mean()) if r.size else 0.0,
        frac_groups_all_equal=(sum(1 for x in with_members if x.max() == x.min()) / len(with_members)
                               if with_members else 0.0),
        mean_reward=float(r.mean()) if r.size else 0.0)


def loss_fwd(H, W, targets, mask, seq_id, group_id, reward, logp_inf,
             S, P, beta_v, beta_loss, loss_scale):
    """Whole forward: token log-probs -> sequence sums -> Eq. 2 -> Eq. 3."""
    lp, lse = token_logprobs(H, W, targets, mask)
    s, D, T = sequence_sums(lp, logp_inf, mask, seq_id, S)
    out = loss_from_sums(D, reward, group_id, P, beta_v, beta_loss, loss_scale)
    out.update(token_logp=lp, lse=lse, seq_logp=s, D=D, T=T)
    return out


# --------------------------------------------------------------------------
# gradient of Eq. 3 with respect to H and W
# --------------------------------------------------------------------------
def loss_bwd(H, W, targets, mask, seq_id, coef):
    """dL/dH [N, d] and dL/dW [V, d].

    With p[n, v] = softmax_v z[n, v] and c_i = dL/ds_i, the chain rule through
    s_i = sum_n m_n (z[n, y_n] - lse_n) gives
        g[n, v] = dL/dz[n, v] = c_{seq(n)} m_n ( [v == y_n] - p[n, v] ),
        dH = g . W,      dW = g^T . H.
    Rows with mask == 0 have g = 0, hence a zero row in dH.
    """
    H = np.asarray(H, dtype=np.float64)
    W = np.asarray(W, dtype=np.float64)
    N, d = H.shape
    mask = np.asarray(mask).astype(bool)
    targets = np.asarray(targets).astype(np.int64)
    seq_id = np.asarray(seq_id).astype(np.int64)
    coef = np.asarray(coef, dtype=np.float64)
    dH = np.zeros((N, d))
    dW = np.zeros_like(W)
    live = np.flatnonzero(mask)
    if live.size == 0:
        return dH, dW
    z = logits(H[live], W)
    l = log_sum_exp(z)
    g = -np.exp(z - l[:, None])
    g[np.arange(live.size), targets[live]] += 1.0
    g *= coef[seq_id[live]][:, None]
    dH[live] = g @ W
    dW = g.T @ H[live]
    return dH, dW


# --------------------------------------------------------------------------
# the paper's baseline: GRPO with token-level importance weights
# (the display in the Background section)
# --------------------------------------------------------------------------
def group_advantage(reward, group_id, P, eps):
    """Normalised advantage A_i = (r_i - mean_p) / (std_p + eps) over the
    members of the rollout's group (population standard deviation)."""
    r = np.asarray(reward, dtype=np.float64)
    g = np.asarray(group_id).astype(np.int64)
    adv = np.zeros_like(r)
    for p in range(P):
        sel = g == p
        if sel.any():
            adv[sel] = (r[sel] - r[sel].mean()) / (r[sel].std() + eps)
    return adv


def grpo_from_logprobs(lp, logp_old, logp_inf, mask, seq_id, adv, S, clip_eps, loss_scale):
    """Loss and per-token coefficients of the importance-weighted GRPO objective.

    Per response token t of rollout i, with r_t = exp(lp_t - lp_old_t) and the
    importance ratio w_t = exp(lp_old_t - lp_inf_t) (data):
        term_t = w_t * min(r_t A_i, clip(r_t, 1 - eps, 1 + eps) A_i)
        loss   = -loss_scale * sum_i (1/|y_i|) sum_t term_t
        c_t    = dloss/dlp_t = -loss_scale/|y_i| * w_t * A_i * r_t on the unclipped
                 branch, 0 on the clipped one (a constant).
    """
    m = np.asarray(mask).astype(bool)
    sid = np.asarray(seq_id).astype(np.int64)
    lp = np.asarray(lp, dtype=np.float64)
    N = lp.shape[0]
    T = np.zeros(S)
    np.add.at(T, sid, m.astype(np.float64))
    coef = np.zeros(N)
    clipped = np.zeros(N, dtype=bool)
    ratio = np.ones(N)
    loss = 0.0
    for n in np.flatnonzero(m):
        i = sid[n]
        A = float(adv[i])
        r = np.exp(lp[n] - float(logp_old[n]))
        w = np.exp(float(logp_old[n]) - float(logp_inf[n]))
        rc = min(max(r, 1.0 - clip_eps), 1.0 + clip_eps)
        un, cl = r * A, rc * A
        ratio[n] = r
        if un <= cl:
            term = un
            coef[n] = -loss_scale / T[i] * w * A * r
        else:
            term = cl
            clipped[n] = True
        loss += -loss_scale / T[i] * w * term
    n_live = int(m.sum())
    return dict(loss=loss, coef=coef, clipped=clipped, ratio=ratio,
                clip_frac=(clipped.sum() / n_live if n_live else 0.0), T=T)


def grpo_fwd(H, W, targets, mask, seq_id, logp_old, logp_inf, adv, S, clip_eps, loss_scale):
    lp, lse = token_logprobs(H, W, targets, mask)
    out = grpo_from_logprobs(lp, logp_old, logp_inf, mask, seq_id, adv, S, clip_eps, loss_scale)
    s, _, _ = sequence_sums(lp, np.zeros_like(lp), mask, seq_id, S)
    out.update(token_logp=lp, lse=lse, seq_logp=s)
    return out


def token_coef_bwd(H, W, targets, mask, coef_tok):
    """dH, dW for a per-token coefficient: g[n, v] = c_n ([v == y_n] - p[n, v])."""
    H = np.asarray(H, dtype=np.float64)
    n = H.shape[0]
    return loss_bwd(H, W, targets, mask, np.arange(n), coef_tok)


# --------------------------------------------------------------------------
# the optimizer step of the paper's hyper-parameter tables: AdamW with
# gradient clipping by norm (decoupled weight decay, Loshchilov & Hutter)
# --------------------------------------------------------------------------
def adamw_step(theta, grad, m, v, step, lr, beta1, beta2, eps, weight_decay, clip_norm, other_sq_norm=0.0):
    """One AdamW step on float64 arrays; returns (theta, m, v, grad_norm).

    The gradient is first scaled by min(1, clip_norm / (||grad|| + 1e-6)) with
    ||grad||^2 = sum(grad^2) + other_sq_norm (clip_norm <= 0: no clipping)."""
    theta = np.asarray(theta, dtype=np.float64)
    g = np.asarray(grad, dtype=np.float64)
    norm = float(np.sqrt((g * g).sum() + other_sq_norm))
    if clip_norm > 0:
        g = g * min(1.0, clip_norm / (norm + 1e-6))
    m = beta1 * np.asarray(m, dtype=np.float64) + (1.0 - beta1) * g
    v = beta2 * np.asarray(v, dtype=np.float64) + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    theta = theta * (1.0 - lr * weight_decay) - lr * mhat / (np.sqrt(vhat) + eps)
    return theta, m, v, norm


def token_entropy(H, W, mask):
    """Per-row policy entropy -sum_v p ln p (the diagnostic tracked in the
    paper's entropy figure); 0 on masked rows."""
    H = np.asarray(H, dtype=np.float64)
    mask = np.asarray(mask).astype(bool)
    ent = np.zeros(H.shape[0])
    live = np.flatnonzero(mask)
    if live.size:
        z = logits(H[live], W)
        l = log_sum_exp(z)
        p = np.exp(z - l[:, None])
        ent[live] = l - (p * z).sum(axis=1)
    return ent


def sequence_entropy(ent, mask, seq_id, S):
    """Per-sequence mean of the token entropies over the response tokens (0 for
    a sequence without any) and the mean over all response tokens of the batch:
    the "sequence entropy" the paper's training-dynamics figure tracks, read as
    the token-level entropy averaged over the response."""
    m = np.asarray(mask).astype(bool)
    seq_id = np.asarray(seq_id).astype(np.int64)
    ent = np.asarray(ent, dtype=np.float64)
    per_seq = np.zeros(S)
    for i in range(S):
        rows = m & (seq_id == i)
        if rows.any():
            per_seq[i] = ent[rows].mean()
    mean = ent[m].mean() if m.any() else 0.0
    return per_seq, float(mean)


def row_entropy(h, W):
    """Entropy of one row's next-token distribution."""
    z = np.asarray(W, dtype=np.float64) @ np.asarray(h, dtype=np.float64)
    M = z.max()
    e = np.exp(z - M)
    lse = M + np.log(e.sum())
    return lse - (e * z).sum() / e.sum()


# --------------------------------------------------------------------------
# one-row / one-vocab-row forms for sampled checks at sizes where the whole
# [N, V] problem is out of reach for a CPU.  Same definitions, one row each.
# --------------------------------------------------------------------------
def row_logprob(h, W, target):
    """(lp, lse) for a single hidden-state row h [d]."""
    z = np.asarray(W, dtype=np.float64) @ np.asarray(h, dtype=np.float64)
    M = z.max()
    lse = M + np.log(np.exp(z - M).sum())
    return z[int(target)] - lse, lse


def row_dH(h, W, target, c):
    """dL/dh for a single live row with sequence coefficient c."""
    W = np.asarray(W, dtype=np.float64)
    z = W @ np.asarray(h, dtype=np.float64)
    M = z.max()
    lse = M + np.log(np.exp(z - M).sum())
    g = -np.exp(z - lse)
    g[int(target)] += 1.0
    return c * (g @ W)


def vocab_rows_dW(vs, W_vs, H, targets, mask, seq_id, coef, lse):
    """Rows vs of dL/dW at once (same definition as vocab_row_dW, one matrix
    product for the logits of those vocabulary rows).  The result is additive
    over row blocks of H, so a caller may sum it over chunks of rows."""
    H = np.asarray(H, dtype=np.float64)
    vs = np.asarray(vs).astype(np.int64)
    m = np.asarray(mask).astype(np.float64)
    Z = H @ np.asarray(W_vs, dtype=np.float64).T                      # [rows, len(vs)]
    P = np.where(m[:, None] > 0, np.exp(Z - np.asarray(lse, dtype=np.float64)[:, None]), 0.0)
    onehot = (np.asarray(targets).astype(np.int64)[:, None] == vs[None, :]).astype(np.float64)
    c = np.asarray(coef, dtype=np.float64)[np.asarray(seq_id).astype(np.int64)] * m
    G = c[:, None] * (onehot - P)
    return G.T @ H


def vocab_row_dW(v, w_v, H, targets, mask, seq_id, coef, lse):
    """dL/dW[v, :] given every live row's log-sum-exp.

    z[n, v] needs only row v of W, so one vocabulary row of dW costs O(N d).
    """
    H = np.asarray(H, dtype=np.float64)
    m = np.asarray(mask).astype(np.float64)
    z_v = H @ np.asarray(w_v, dtype=np.float64)
    p_v = np.where(m > 0, np.exp(z_v - np.asarray(lse, dtype=np.float64)), 0.0)
    onehot = (np.asarray(targets).astype(np.int64) == int(v)).astype(np.float64)
    g_v = np.asarray(coef, dtype=np.float64)[np.asarray(seq_id).astype(np.int64)] * m * (onehot - p_v)
    return g_v @ H

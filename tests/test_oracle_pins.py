"""Pins of the fp64 oracle against what the paper and the mathematics fix.

None of these re-types the oracle's formulas with the same library call: each
is a brute-force loop, a closed form, a limit the paper states, an invariant,
a different library routine, or a finite difference.
"""
import decimal
import math
import os

import numpy as np
import pytest
import scipy.special

from oracle import oapl_oracle as orc

RNG = np.random.default_rng(1234)


def _tiny(N=7, d=5, V=11, S=3, seed=0):
    r = np.random.default_rng(seed)
    H = r.normal(size=(N, d))
    W = r.normal(size=(V, d)) * 0.7
    targets = r.integers(0, V, size=N)
    mask = np.ones(N, dtype=np.uint8)
    mask[2] = 0
    seq_id = np.sort(r.integers(0, S, size=N))
    return H, W, targets, mask, seq_id


# ---------------------------------------------------------------- logits / lse
def test_logits_match_explicit_loops():
    H, W, targets, mask, _ = _tiny()
    N, d = H.shape
    V = W.shape[0]
    lp, lse = orc.token_logprobs(H, W, targets, mask)
    for n in range(N):
        if not mask[n]:
            assert lp[n] == 0.0 and lse[n] == 0.0
            continue
        z = [sum(H[n, k] * W[v, k] for k in range(d)) for v in range(V)]
        tot = sum(math.exp(zv) for zv in z)          # naive, unshifted
        assert lp[n] == pytest.approx(z[targets[n]] - math.log(tot), abs=1e-12)
        assert lse[n] == pytest.approx(math.log(tot), abs=1e-12)


def test_softmax_rows_sum_to_one():
    H, W, _, _, _ = _tiny(N=4, V=13)
    V = W.shape[0]
    for n in range(H.shape[0]):
        Hn = np.repeat(H[n:n + 1], V, axis=0)
        lp, _ = orc.token_logprobs(Hn, W, np.arange(V), np.ones(V, dtype=np.uint8))
        assert abs(np.exp(lp).sum() - 1.0) < 1e-12


def test_zero_weight_gives_uniform():
    H, W, targets, mask, _ = _tiny(V=17)
    lp, lse = orc.token_logprobs(H, np.zeros_like(W), targets, mask)
    live = mask.astype(bool)
    assert np.allclose(lp[live], -math.log(17), atol=1e-14)
    lp2, _ = orc.token_logprobs(np.zeros_like(H), W, targets, mask)
    assert np.allclose(lp2[live], -math.log(17), atol=1e-14)


def test_two_token_vocab_is_logistic():
    r = np.random.default_rng(3)
    H = r.normal(size=(6, 4))
    W = r.normal(size=(2, 4))
    t = r.integers(0, 2, size=6)
    lp, _ = orc.token_logprobs(H, W, t, np.ones(6, dtype=np.uint8))
    for n in range(6):
        z = W @ H[n]
        other = z[1 - t[n]] - z[t[n]]
        assert lp[n] == pytest.approx(-math.log1p(math.exp(other)), abs=1e-13)


def test_against_scipy_log_softmax_and_large_logits():
    r = np.random.default_rng(5)
    H = r.normal(size=(9, 8)) * 40.0          # logits of magnitude ~100: needs the max shift
    W = r.normal(size=(33, 8))
    t = r.integers(0, 33, size=9)
    lp, lse = orc.token_logprobs(H, W, t, np.ones(9, dtype=np.uint8))
    z = np.einsum("nk,vk->nv", H, W)
    ref = scipy.special.log_softmax(z, axis=1)
    assert np.allclose(lp, ref[np.arange(9), t], atol=1e-10)
    assert np.allclose(lse, scipy.special.logsumexp(z, axis=1), atol=1e-10)
    assert np.all(np.isfinite(lp))


def test_bf16_widening_is_exact():
    import torch
    x = torch.randn(1000, dtype=torch.float32).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(orc.bf16_bits_to_f64(bits), x.to(torch.float64).numpy())


def test_sequence_sums_by_loop_and_nan_in_masked_rows():
    r = np.random.default_rng(7)
    N, S = 40, 5
    lp = r.normal(size=N)
    q = r.normal(size=N)
    mask = (r.random(N) < 0.7).astype(np.uint8)
    q[mask == 0] = np.nan
    seq_id = np.sort(r.integers(0, S, size=N))
    s, D, T = orc.sequence_sums(lp, q, mask, seq_id, S)
    for i in range(S):
        idx = [n for n in range(N) if seq_id[n] == i and mask[n]]
        assert s[i] == pytest.approx(sum(lp[n] for n in idx), abs=1e-12)
        assert D[i] == pytest.approx(sum(lp[n] - q[n] for n in idx), abs=1e-12)
        assert T[i] == len(idx)


# ---------------------------------------------------------------- Eq. 2
def test_value_equal_rewards_and_singleton():
    v = orc.value_estimate([0.7] * 8 + [3.0], [0] * 8 + [1], 3, 0.37)
    assert v[0] == pytest.approx(0.7, abs=1e-15)
    assert v[1] == pytest.approx(3.0, abs=1e-15)
    assert v[2] == 0.0                                    # empty group


def test_value_limits_stated_by_the_paper():
    r = RNG.random(8)
    g = np.zeros(8, dtype=int)
    assert orc.value_estimate(r, g, 1, 1e-4)[0] == pytest.approx(r.max(), abs=1e-3)
    assert orc.value_estimate(r, g, 1, 1e7)[0] == pytest.approx(r.mean(), abs=1e-6)


def test_value_binary_closed_form():
    for beta in (0.1, 0.5, 1.0, 2.0, 10.0):
        for k in range(0, 9):
            r = np.array([1.0] * k + [0.0] * (8 - k))
            want = beta * math.log(1.0 + (k / 8.0) * math.expm1(1.0 / beta))
            got = orc.value_estimate(r, np.zeros(8, dtype=int), 1, beta)[0]
            assert got == pytest.approx(want, rel=1e-12, abs=1e-13)


def test_value_literal_formula_in_decimal_arithmetic():
    decimal.getcontext().prec = 60
    r = [0.0, 1.0, 1.0, 0.0, 0.25, 1.0, 0.0, 0.5]
    for beta in (1e-3, 1e-2, 0.3, 1.0, 5.0):
        tot = sum((decimal.Decimal(x) / decimal.Decimal(beta)).exp() for x in r)
        want = float(decimal.Decimal(beta) * (tot / len(r)).ln())
        got = orc.value_estimate(r, np.zeros(len(r), dtype=int), 1, beta)[0]
        assert got == pytest.approx(want, rel=1e-12)


def test_value_shift_bounds_monotone_and_scattered_groups():
    r = RNG.normal(size=12)
    g = np.array([0, 1, 2] * 4)                          # members not adjacent
    v = orc.value_estimate(r, g, 3, 0.8)
    v_shift = orc.value_estimate(r + 2.5, g, 3, 0.8)
    assert np.allclose(v_shift, v + 2.5, atol=1e-13)
    prev = None
    for beta in (0.05, 0.2, 1.0, 4.0, 50.0):
        vb = orc.value_estimate(r, g, 3, beta)
        for p in range(3):
            rp = r[g == p]
            assert rp.mean() - 1e-12 <= vb[p] <= rp.max() + 1e-12
        if prev is not None:
            assert np.all(vb <= prev + 1e-12)            # non-increasing in beta
        prev = vb


# ---------------------------------------------------------------- Eq. 3
def _problem(seed=0, N=24, d=6, V=19, S=6, P=2):
    r = np.random.default_rng(seed)
    H = r.normal(size=(N, d))
    W = r.normal(size=(V, d)) * 0.5
    targets = r.integers(0, V, size=N)
    mask = (r.random(N) < 0.8).astype(np.uint8)
    seq_id = np.sort(np.concatenate([np.arange(S), r.integers(0, S, size=N - S)]))
    group_id = np.arange(S) % P
    reward = (r.random(S) < 0.5).astype(np.float64)
    logp_inf = r.normal(size=N) - 3.0
    return dict(H=H, W=W, targets=targets, mask=mask, seq_id=seq_id, group_id=group_id,
                reward=reward, logp_inf=logp_inf, S=S, P=P)


def _fwd(p, beta_v=1.0, beta_loss=0.7, lam=1.0):
    return orc.loss_fwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], p["group_id"],
                        p["reward"], p["logp_inf"], p["S"], p["P"], beta_v, beta_loss, lam)


def test_loss_is_the_literal_double_sum():
    p = _problem()
    beta_v, beta_loss = 1.3, 0.4
    out = _fwd(p, beta_v, beta_loss, 1.0)
    lp, _ = orc.token_logprobs(p["H"], p["W"], p["targets"], p["mask"])
    total = 0.0
    for x in range(p["P"]):
        members = [i for i in range(p["S"]) if p["group_id"][i] == x]
        vhat = beta_v * math.log(sum(math.exp(p["reward"][i] / beta_v) for i in members) / len(members))
        for i in members:
            rows = [n for n in range(len(lp)) if p["seq_id"][n] == i and p["mask"][n]]
            ln_pi = sum(lp[n] for n in rows)
            ln_pi_inf = sum(p["logp_inf"][n] for n in rows)
            total += (beta_loss * (ln_pi - ln_pi_inf) - (p["reward"][i] - vhat)) ** 2
    assert out["loss"] == pytest.approx(total, rel=1e-12)


def test_zero_loss_and_zero_gradient_at_the_optimum():
    # If beta ln(pi/pi_vllm) already equals r - V^ for every rollout, Eq. 3 is 0.
    p = _problem(seed=2)
    beta_v, beta_loss = 1.0, 0.5
    first = _fwd(p, beta_v, beta_loss)
    lp = first["token_logp"]
    q = p["logp_inf"].copy()
    for i in range(p["S"]):
        rows = np.flatnonzero((p["seq_id"] == i) & (p["mask"] == 1))
        assert rows.size > 0
        want_D = first["A"][i] / beta_loss
        q[rows] = lp[rows]
        q[rows[0]] -= want_D
    p["logp_inf"] = q
    out = _fwd(p, beta_v, beta_loss)
    assert out["loss"] < 1e-24
    dH, dW = orc.loss_bwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], out["coef"])
    assert np.abs(dH).max() < 1e-10 and np.abs(dW).max() < 1e-10


def test_loss_scalings():
    p = _problem(seed=4)
    a = _fwd(p, 1.0, 0.7, 1.0)["loss"]
    b = _fwd(p, 1.0, 0.7, 1.0 / p["S"])["loss"]
    assert b == pytest.approx(a / p["S"], rel=1e-13)
    p["reward"][:] = 1.0                                   # A = 0: loss = lam * beta^2 * sum D^2
    c = _fwd(p, 1.0, 0.7, 1.0)
    d = _fwd(p, 1.0, 1.4, 1.0)
    assert np.allclose(c["A"], 0.0, atol=1e-15)
    assert d["loss"] == pytest.approx(4.0 * c["loss"], rel=1e-12)
    assert c["loss"] == pytest.approx(0.49 * np.sum(c["D"] ** 2), rel=1e-12)


def test_paper_hyperparameters_fixture():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_hparams.txt")
    kv = {}
    for line in open(path):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            kv[k] = v
    beta_v, beta_loss, G = float(kv["beta_v"][0]), float(kv["beta_loss"][0]), int(kv["generations_per_prompt"][0])
    assert (beta_v, beta_loss, G) == (1.0, 1e-3, 8)
    # with those temperatures and k of 8 binary rewards correct
    r = np.array([1, 0, 0, 1, 0, 0, 0, 1], dtype=float)
    v = orc.value_estimate(r, np.zeros(8, dtype=int), 1, beta_v)[0]
    assert v == pytest.approx(math.log(1 + 3 / 8 * (math.e - 1)), rel=1e-13)


# ---------------------------------------------------------------- gradient
def test_gradient_matches_central_differences():
    p = _problem(seed=9, N=18, d=4, V=9, S=4, P=2)
    beta_v, beta_loss, lam = 0.9, 0.6, 0.25
    out = _fwd(p, beta_v, beta_loss, lam)
    dH, dW = orc.loss_bwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], out["coef"])
    h = 1e-6
    for name, grad in (("H", dH), ("W", dW)):
        base = p[name]
        for idx in np.ndindex(*base.shape):
            q = dict(p)
            plus, minus = base.copy(), base.copy()
            plus[idx] += h
            minus[idx] -= h
            q[name] = plus
            lp_ = _fwd(q, beta_v, beta_loss, lam)["loss"]
            q[name] = minus
            lm_ = _fwd(q, beta_v, beta_loss, lam)["loss"]
            fd = (lp_ - lm_) / (2 * h)
            assert grad[idx] == pytest.approx(fd, rel=2e-6, abs=2e-7), (name, idx)


def test_gradient_invariants():
    p = _problem(seed=11)
    out = _fwd(p)
    dH, dW = orc.loss_bwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], out["coef"])
    assert np.abs(dW.sum(axis=0)).max() < 1e-12          # rows of g sum to 0
    assert np.all(dH[p["mask"] == 0] == 0.0)
    dH0, _ = orc.loss_bwd(p["H"], np.zeros_like(p["W"]), p["targets"], p["mask"], p["seq_id"], out["coef"])
    assert np.all(dH0 == 0.0)
    never = [v for v in range(p["W"].shape[0]) if v not in set(p["targets"][p["mask"] == 1])]
    z = p["H"] @ p["W"].T
    prob = np.exp(z - out["lse"][:, None])
    for v in never[:3]:
        want = -sum(out["coef"][p["seq_id"][n]] * prob[n, v] * p["H"][n]
                    for n in range(len(z)) if p["mask"][n])
        assert np.allclose(dW[v], want, atol=1e-12)


def test_sampled_forms_agree_with_full_forms():
    p = _problem(seed=13)
    out = _fwd(p)
    dH, dW = orc.loss_bwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], out["coef"])
    for n in np.flatnonzero(p["mask"])[:5]:
        lp, lse = orc.row_logprob(p["H"][n], p["W"], p["targets"][n])
        assert lp == pytest.approx(out["token_logp"][n], abs=1e-12)
        g = orc.row_dH(p["H"][n], p["W"], p["targets"][n], out["coef"][p["seq_id"][n]])
        assert np.allclose(g, dH[n], atol=1e-12)
    for v in (0, 5, 18):
        row = orc.vocab_row_dW(v, p["W"][v], p["H"], p["targets"], p["mask"], p["seq_id"],
                               out["coef"], out["lse"])
        assert np.allclose(row, dW[v], atol=1e-12)
    vs = [0, 5, 18, 3]
    full = orc.vocab_rows_dW(vs, p["W"][vs], p["H"], p["targets"], p["mask"], p["seq_id"], out["coef"], out["lse"])
    assert np.allclose(full, dW[vs], atol=1e-12)
    half = len(p["mask"]) // 2                                           # additive over row blocks
    parts = sum(orc.vocab_rows_dW(vs, p["W"][vs], p["H"][sl], p["targets"][sl], p["mask"][sl], p["seq_id"][sl],
                                  out["coef"], out["lse"][sl]) for sl in (slice(0, half), slice(half, None)))
    assert np.allclose(parts, dW[vs], atol=1e-12)


def test_entropy_definition():
    H, W, _, mask, _ = _tiny()
    ent = orc.token_entropy(H, W, mask)
    for n in range(H.shape[0]):
        if not mask[n]:
            assert ent[n] == 0.0
            continue
        z = W @ H[n]
        pr = np.exp(z) / np.exp(z).sum()
        assert ent[n] == pytest.approx(-(pr * np.log(pr)).sum(), abs=1e-12)
    assert orc.token_entropy(H, np.zeros_like(W), mask)[0] == pytest.approx(math.log(W.shape[0]))


def test_entropy_closed_forms_bounds_and_scipy():
    import scipy.stats
    r = np.random.default_rng(7)
    # two-token vocabulary: binary entropy of the logistic of the logit gap
    H = r.normal(size=(6, 4))
    W = r.normal(size=(2, 4))
    ent = orc.token_entropy(H, W, np.ones(6, dtype=np.uint8))
    gap = H @ (W[0] - W[1])
    q = 1.0 / (1.0 + np.exp(-gap))
    assert np.allclose(ent, -(q * np.log(q) + (1 - q) * np.log1p(-q)), atol=1e-12)
    # a different library routine on explicit probabilities; bounds; one-hot limit
    H, W, _, mask, seq_id = _tiny(N=9, d=6, V=13, S=3, seed=3)
    ent = orc.token_entropy(H, W, mask)
    p = scipy.special.softmax(H @ W.T, axis=1)
    want = scipy.stats.entropy(p, axis=1)
    assert np.allclose(ent[mask == 1], want[mask == 1], atol=1e-12)
    assert np.all(ent >= 0) and np.all(ent <= math.log(13) + 1e-12)
    assert orc.token_entropy(50.0 * H, W, mask).max() < ent.max()          # sharper logits, lower entropy
    assert orc.row_entropy(H[0], W) == pytest.approx(ent[0], abs=1e-12)
    # per-sequence and batch means by explicit loops
    per_seq, mean = orc.sequence_entropy(ent, mask, seq_id, 3)
    tot, cnt = 0.0, 0
    for i in range(3):
        vals = [ent[n] for n in range(9) if mask[n] and seq_id[n] == i]
        assert per_seq[i] == pytest.approx(sum(vals) / len(vals) if vals else 0.0, abs=1e-14)
        tot, cnt = tot + sum(vals), cnt + len(vals)
    assert mean == pytest.approx(tot / cnt, abs=1e-14)
    assert orc.sequence_entropy(ent, np.zeros(9, dtype=np.uint8), seq_id, 3)[1] == 0.0


# ---------------------------------------------------------------- GRPO baseline
def _grpo_problem(seed=0, noise=0.15):
    r = np.random.default_rng(seed)
    N, d, V, S, P = 14, 5, 9, 4, 2
    H = r.normal(size=(N, d))
    W = r.normal(size=(V, d)) * 0.6
    targets = r.integers(0, V, size=N)
    seq_id = np.sort(np.concatenate([np.arange(S), r.integers(0, S, size=N - S)]))
    mask = np.ones(N, dtype=np.uint8)
    for i in (0, 2):                       # a masked row in two sequences that keep other rows
        rows = np.flatnonzero(seq_id == i)
        if len(rows) > 1:
            mask[rows[0]] = 0
    mask[np.flatnonzero(seq_id == np.bincount(seq_id).argmax())[-1]] = 0
    group_id = np.array([0, 0, 1, 1])
    reward = np.array([1.0, 0.0, 0.5, 2.0])
    lp, _ = orc.token_logprobs(H, W, targets, mask)
    logp_old = lp + noise * r.normal(size=N)
    logp_inf = logp_old + 0.1 * r.normal(size=N)
    return dict(H=H, W=W, targets=targets, mask=mask, seq_id=seq_id, group_id=group_id, reward=reward,
                logp_old=logp_old, logp_inf=logp_inf, S=S, P=P)


def test_group_advantage_is_standardised_within_groups():
    r = np.array([1.0, 0.0, 0.0, 1.0, 3.0, 3.0, 3.0, 7.0])
    g = np.array([0, 0, 0, 0, 1, 1, 1, 2])
    adv = orc.group_advantage(r, g, 4, 0.0 + 1e-12)
    assert abs(adv[:4].mean()) < 1e-9 and adv[:4].std() == pytest.approx(1.0, abs=1e-9)
    assert np.all(adv[4:7] == 0.0) and adv[7] == 0.0                  # equal rewards, singleton
    # invariance to a positive affine map of the rewards (eps = 0 in the limit)
    adv2 = orc.group_advantage(5.0 * r - 3.0, g, 4, 1e-12)
    assert np.allclose(adv, adv2, atol=1e-9)
    assert orc.group_advantage(r, g, 4, 1.0)[0] == pytest.approx(0.5 / (0.5 + 1.0))


def test_grpo_loss_is_the_literal_display():
    p = _grpo_problem(1, noise=0.3)
    adv = orc.group_advantage(p["reward"], p["group_id"], p["P"], 1e-6)
    out = orc.grpo_fwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], p["logp_old"], p["logp_inf"],
                       adv, p["S"], 0.2, 0.25)
    # the display, typed out: 1/|y| sum_t  IS ratio * min(r A, clip(r) A), summed over rollouts
    z = p["H"] @ p["W"].T
    lsm = z - scipy.special.logsumexp(z, axis=1, keepdims=True)
    J = 0.0
    for i in range(p["S"]):
        rows = [n for n in range(len(p["mask"])) if p["mask"][n] and p["seq_id"][n] == i]
        acc = 0.0
        for n in rows:
            pi, pi_old, pi_vllm = (math.exp(lsm[n, p["targets"][n]]), math.exp(p["logp_old"][n]),
                                   math.exp(p["logp_inf"][n]))
            r_t = pi / pi_old
            acc += (pi_old / pi_vllm) * min(r_t * adv[i], float(np.clip(r_t, 0.8, 1.2)) * adv[i])
        J += acc / len(rows)
    assert out["loss"] == pytest.approx(-0.25 * J, rel=1e-12)
    assert 0 < out["clipped"].sum() < p["mask"].sum()                 # both branches are exercised


def test_grpo_on_policy_reduces_to_the_policy_gradient():
    # pi_old = pi and pi_vllm = pi_old: every ratio is 1, nothing is clipped, the loss is
    # -lambda sum_i A_i (zero for standardised advantages) and dloss/dlp_t = -lambda A_i / |y_i|
    p = _grpo_problem(2)
    lp, _ = orc.token_logprobs(p["H"], p["W"], p["targets"], p["mask"])
    adv = orc.group_advantage(p["reward"], p["group_id"], p["P"], 1e-9)
    out = orc.grpo_from_logprobs(lp, lp, lp, p["mask"], p["seq_id"], adv, p["S"], 0.2, 1.0)
    assert abs(out["loss"]) < 1e-9 and not out["clipped"].any()
    for n in np.flatnonzero(p["mask"]):
        i = p["seq_id"][n]
        assert out["coef"][n] == pytest.approx(-adv[i] / out["T"][i], rel=1e-12)


def test_grpo_clipped_tokens_are_constant():
    p = _grpo_problem(3, noise=0.0)
    lp, _ = orc.token_logprobs(p["H"], p["W"], p["targets"], p["mask"])
    adv = np.array([1.0, -1.0, 1.0, -1.0])
    old = lp.copy()
    old[p["seq_id"] == 0] -= 0.5       # r = e^0.5 > 1.2 with A > 0: clipped at (1+eps) A
    old[p["seq_id"] == 1] += 0.5       # r = e^-0.5 < 0.8 with A < 0: clipped at (1-eps) A
    old[p["seq_id"] == 2] += 0.5       # r < 0.8 with A > 0: unclipped
    old[p["seq_id"] == 3] -= 0.5       # r > 1.2 with A < 0: unclipped
    out = orc.grpo_from_logprobs(lp, old, old, p["mask"], p["seq_id"], adv, p["S"], 0.2, 1.0)
    live = p["mask"].astype(bool)
    assert out["clipped"][live & (p["seq_id"] <= 1)].all() and not out["clipped"][live & (p["seq_id"] >= 2)].any()
    assert np.all(out["coef"][p["seq_id"] <= 1] == 0.0)
    want = -(1.2 * 1.0 + 0.8 * -1.0 + math.exp(-0.5) * 1.0 + math.exp(0.5) * -1.0)
    assert out["loss"] == pytest.approx(want, rel=1e-12)


def test_grpo_gradient_matches_central_differences():
    p = _grpo_problem(4)
    adv = orc.group_advantage(p["reward"], p["group_id"], p["P"], 1e-6)
    f = lambda H, W: orc.grpo_fwd(H, W, p["targets"], p["mask"], p["seq_id"], p["logp_old"], p["logp_inf"],
                                  adv, p["S"], 0.2, 0.5)
    out = f(p["H"], p["W"])
    assert np.abs(np.abs(out["ratio"][p["mask"] == 1] - 1.0) - 0.2).min() > 1e-3   # away from the kinks
    dH, dW = orc.token_coef_bwd(p["H"], p["W"], p["targets"], p["mask"], out["coef"])
    h = 1e-6
    for X, dX, name in ((p["H"], dH, "H"), (p["W"], dW, "W")):
        for idx in np.ndindex(X.shape):
            Xp, Xm = X.copy(), X.copy()
            Xp[idx] += h
            Xm[idx] -= h
            num = ((f(Xp, p["W"]) if name == "H" else f(p["H"], Xp))["loss"] -
                   (f(Xm, p["W"]) if name == "H" else f(p["H"], Xm))["loss"]) / (2 * h)
            assert num == pytest.approx(dX[idx], rel=2e-5, abs=2e-8), (name, idx)
    assert np.all(dH[p["mask"] == 0] == 0.0)


# ---------------------------------------------------------------- AdamW + clipping by norm
def test_adamw_matches_torch_optimizer_and_clip_grad_norm():
    import torch
    r = np.random.default_rng(11)
    theta0 = r.normal(size=(37,)) * 0.02
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=1e-2)
    p = torch.nn.Parameter(torch.tensor(theta0, dtype=torch.float64))
    opt = torch.optim.AdamW([p], lr=hp["lr"], betas=(hp["beta1"], hp["beta2"]), eps=hp["eps"],
                            weight_decay=hp["weight_decay"])
    theta, m, v = theta0.copy(), np.zeros(37), np.zeros(37)
    for step in range(1, 6):
        g = r.normal(size=37) * (10.0 if step % 2 else 1e-3)       # clipped and unclipped steps
        p.grad = torch.tensor(g, dtype=torch.float64)
        torch.nn.utils.clip_grad_norm_([p], max_norm=1.0)
        opt.step()
        theta, m, v, norm = orc.adamw_step(theta, g, m, v, step, clip_norm=1.0, **hp)
        assert norm == pytest.approx(np.linalg.norm(g), rel=1e-14)
        assert np.allclose(theta, p.detach().numpy(), rtol=1e-12, atol=1e-15)


def test_adamw_closed_forms():
    g = np.array([3.0, -0.5, 2.0, -4.0])
    th = np.array([1.0, -2.0, 0.5, 0.25])
    z = np.zeros(4)
    # first step, no decay, eps = 0: the bias-corrected ratio is sign(g), whatever the gradient's scale,
    # so clipping cannot change it
    a, _, _, _ = orc.adamw_step(th, g, z, z, 1, 1e-2, 0.9, 0.95, 0.0, 0.0, 0.0)
    assert np.allclose(a, th - 1e-2 * np.sign(g), atol=1e-15)
    b, _, _, _ = orc.adamw_step(th, g, z, z, 1, 1e-2, 0.9, 0.95, 0.0, 0.0, 1e-3)
    assert np.allclose(a, b, atol=1e-12)
    # zero gradient: decoupled weight decay only
    c, m, v, norm = orc.adamw_step(th, z, z, z, 1, 1e-2, 0.9, 0.95, 1e-8, 0.1, 1.0)
    assert np.allclose(c, th * (1 - 1e-3), atol=1e-15) and norm == 0.0 and not m.any() and not v.any()
    # the clipped gradient has norm clip_norm (up to the 1e-6 guard): read it off m after one step
    _, m, _, norm = orc.adamw_step(th, g, z, z, 1, 1e-2, 0.9, 0.95, 1e-8, 0.0, 0.5)
    assert np.linalg.norm(m / 0.1) == pytest.approx(0.5, rel=1e-5) and norm == pytest.approx(np.linalg.norm(g))
    # other parameters' gradient norm enters the clip factor
    _, m2, _, norm2 = orc.adamw_step(th, g, z, z, 1, 1e-2, 0.9, 0.95, 1e-8, 0.0, 0.5, other_sq_norm=100.0)
    assert norm2 == pytest.approx(math.sqrt((g * g).sum() + 100.0))
    assert np.allclose(m2, 0.1 * g * 0.5 / (norm2 + 1e-6), rtol=1e-12)


# ---------------------------------------------------------------- autograd as an independent route
def test_gradients_match_torch_autograd():
    # Eq. 3 and the GRPO display typed out with torch ops in fp64 and differentiated by autograd:
    # a different library and a different route (reverse mode through log_softmax) to dH and dW
    import torch
    p = _grpo_problem(5, noise=0.3)
    Ht = torch.tensor(p["H"], dtype=torch.float64, requires_grad=True)
    Wt = torch.tensor(p["W"], dtype=torch.float64, requires_grad=True)
    tg = torch.tensor(p["targets"], dtype=torch.int64)
    m = torch.tensor(p["mask"], dtype=torch.float64)
    sid = torch.tensor(p["seq_id"], dtype=torch.int64)
    lp = torch.log_softmax(Ht @ Wt.T, dim=1).gather(1, tg[:, None]).squeeze(1)

    # OAPL: sum_i (beta2 * sum_t m (lp - q) - (r_i - vhat_g(i)))^2 with vhat from Eq. 2
    beta_v, beta_loss, lam = 0.7, 0.3, 0.25
    q = torch.tensor(p["logp_inf"], dtype=torch.float64)
    r = torch.tensor(p["reward"], dtype=torch.float64)
    gid = torch.tensor(p["group_id"], dtype=torch.int64)
    D = torch.zeros(p["S"], dtype=torch.float64).index_add(0, sid, m * (lp - q))
    vhat = torch.stack([beta_v * torch.log(torch.mean(torch.exp(r[gid == g] / beta_v))) for g in range(p["P"])])
    loss = lam * torch.sum((beta_loss * D - (r - vhat[gid])) ** 2)
    gH, gW = torch.autograd.grad(loss, (Ht, Wt), retain_graph=True)
    out = orc.loss_fwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], p["group_id"], p["reward"],
                       p["logp_inf"], p["S"], p["P"], beta_v, beta_loss, lam)
    dH, dW = orc.loss_bwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], out["coef"])
    assert out["loss"] == pytest.approx(float(loss.detach()), rel=1e-12)
    assert np.allclose(dH, gH.numpy(), rtol=1e-9, atol=1e-12) and np.allclose(dW, gW.numpy(), rtol=1e-9, atol=1e-12)

    # GRPO: -lam * sum_i 1/|y_i| sum_t w_t min(r_t A_i, clip(r_t) A_i), w_t detached data
    adv = torch.tensor(orc.group_advantage(p["reward"], p["group_id"], p["P"], 1e-6))
    old = torch.tensor(p["logp_old"], dtype=torch.float64)
    ratio = torch.exp(lp - old)
    w = torch.exp(old - q)
    A = adv[sid]
    T = torch.zeros(p["S"], dtype=torch.float64).index_add(0, sid, m)
    term = w * torch.minimum(ratio * A, torch.clamp(ratio, 0.8, 1.2) * A) * m / T[sid]
    gloss = -lam * term.sum()
    gH, gW = torch.autograd.grad(gloss, (Ht, Wt))
    go = orc.grpo_fwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], p["logp_old"], p["logp_inf"],
                      adv.numpy(), p["S"], 0.2, lam)
    dH, dW = orc.token_coef_bwd(p["H"], p["W"], p["targets"], p["mask"], go["coef"])
    assert go["loss"] == pytest.approx(float(gloss.detach()), rel=1e-12)
    assert go["clipped"].any()
    assert np.allclose(dH, gH.numpy(), rtol=1e-9, atol=1e-12) and np.allclose(dW, gW.numpy(), rtol=1e-9, atol=1e-12)


# --------------------------------------------------------------------------
# batch diagnostics
# --------------------------------------------------------------------------
def test_batch_stats_on_a_hand_computed_example():
    # four rollouts in two groups; the third has no response token and must not count in the
    # log-ratio statistics; group 1 has all-equal rewards
    D = [1.0, -3.0, 123.0, 2.0]
    T = [2, 1, 0, 4]
    st = orc.batch_stats(D, T, reward=[1.0, 0.0, 1.0, 1.0], group_id=[0, 0, 1, 1], vhat=[0.7, 1.0], P=3)
    assert st["live_tokens"] == 7.0
    assert st["mean_abs_log_ratio"] == pytest.approx(2.0, rel=1e-15)       # (1 + 3 + 2) / 3
    assert st["max_abs_log_ratio"] == 3.0
    assert st["mean_token_log_ratio"] == pytest.approx(0.0, abs=1e-15)     # (1 - 3 + 2) / 7
    assert st["mean_advantage"] == pytest.approx(-0.1, rel=1e-12)          # (0.3 - 0.7 + 0 + 0) / 4
    assert st["frac_groups_all_equal"] == 0.5                              # the empty third group is not counted
    assert st["mean_reward"] == 0.75


def test_batch_stats_mean_advantage_is_never_positive_with_the_value_estimate_of_eq2():
    # V^ is a log-mean-exp, so V^_p >= mean of the group's rewards (Jensen): the advantages of a
    # group sum to at most 0, with equality exactly when its rewards are all equal
    rng = np.random.default_rng(3)
    for beta in (0.1, 1.0, 10.0):
        r = rng.normal(size=40)
        g = rng.integers(0, 6, size=40)
        vhat = orc.value_estimate(r, g, 7, beta)
        st = orc.batch_stats(np.zeros(40), np.ones(40), r, g, vhat, 7)
        assert st["mean_advantage"] < 0.0
        assert st["frac_groups_all_equal"] <= 1.0 / 6 + 1e-12             # only a one-member group can be "equal"
    r = np.repeat(rng.normal(size=5), 4)                                   # every group constant
    g = np.repeat(np.arange(5), 4)
    st = orc.batch_stats(np.zeros(20), np.ones(20), r, g, orc.value_estimate(r, g, 5, 0.5), 5)
    assert st["mean_advantage"] == pytest.approx(0.0, abs=1e-12) and st["frac_groups_all_equal"] == 1.0


def test_batch_stats_of_an_empty_batch_are_zero():
    st = orc.batch_stats(np.zeros(3), np.zeros(3), np.zeros(3), np.zeros(3, dtype=int), np.zeros(1), 1)
    assert st["live_tokens"] == 0 and st["mean_abs_log_ratio"] == 0 and st["mean_token_log_ratio"] == 0


# --------------------------------------------------------------------------
# symmetries of the softmax LM head (index mistakes break them)
# --------------------------------------------------------------------------
def _step(p, beta_v=0.9, beta_loss=0.6, lam=0.5):
    out = _fwd(p, beta_v, beta_loss, lam)
    dH, dW = orc.loss_bwd(p["H"], p["W"], p["targets"], p["mask"], p["seq_id"], out["coef"])
    return out, dH, dW


def test_adding_one_vector_to_every_row_of_W_changes_nothing():
    # every logit of a row moves by the same h . u, so the next-token distribution, the loss and g are
    # unchanged; rows of g sum to zero, so dH = g.(W + 1 u^T) = g.W, and dW = g^T.H does not see W
    p = _problem(seed=21)
    u = np.random.default_rng(5).normal(size=p["W"].shape[1])
    q = dict(p, W=p["W"] + u[None, :])
    (a, dHa, dWa), (b, dHb, dWb) = _step(p), _step(q)
    assert np.allclose(a["token_logp"], b["token_logp"], atol=1e-12)
    assert a["loss"] == pytest.approx(b["loss"], rel=1e-11)
    assert np.allclose(dHa, dHb, atol=1e-11) and np.allclose(dWa, dWb, atol=1e-11)


def test_permuting_the_vocabulary_permutes_dW_and_nothing_else():
    p = _problem(seed=22)
    V = p["W"].shape[0]
    perm = np.random.default_rng(6).permutation(V)          # new row j holds old row perm[j]
    inv = np.argsort(perm)
    q = dict(p, W=p["W"][perm], targets=inv[p["targets"]])
    (a, dHa, dWa), (b, dHb, dWb) = _step(p), _step(q)
    assert np.allclose(a["token_logp"], b["token_logp"], atol=1e-12)
    assert a["loss"] == pytest.approx(b["loss"], rel=1e-12)
    assert np.allclose(dHa, dHb, atol=1e-12)
    assert np.allclose(dWa[perm], dWb, atol=1e-12)


def test_renumbering_the_groups_and_scaling_the_loss():
    # Eq. 2 / Eq. 3 see a group only as a set of rollouts: renumbering the groups changes nothing;
    # the loss and both gradients are linear in loss_scale
    p = _problem(seed=23, S=8, P=3)
    q = dict(p, group_id=(2 - p["group_id"]))
    (a, dHa, dWa), (b, dHb, dWb) = _step(p), _step(q)
    assert a["loss"] == pytest.approx(b["loss"], rel=1e-13)
    assert np.allclose(a["vhat"], b["vhat"][::-1], atol=1e-13)
    assert np.allclose(dHa, dHb, atol=1e-13) and np.allclose(dWa, dWb, atol=1e-13)
    c, dHc, dWc = _step(p, lam=1.5)
    assert c["loss"] == pytest.approx(3.0 * a["loss"], rel=1e-13)
    assert np.allclose(dHc, 3.0 * dHa, atol=1e-13) and np.allclose(dWc, 3.0 * dWa, atol=1e-13)

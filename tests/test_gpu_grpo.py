"""The importance-weighted GRPO objective (oapl_grpo_loss_fwd_bwd, oapl_group_advantage) against
the fp64 oracle, through the C ABI.

The branch of min(r A, clip(r) A) a token takes is a floating-point comparison that decides
between a full and a zero coefficient.  The library takes it on fp32 log-probabilities that
carry up to 2e-3 of error, the oracle in fp64, so the inputs keep every ratio at least 1e-2
away from the two clip boundaries; what is compared is then unique.

Tolerances: token log-probs 2e-3; gradients 1e-2 relative Frobenius; the loss is a signed sum
that cancels (standardised advantages sum to zero per group), so its 1e-3 is relative to the
sum of the absolute per-token terms."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu
CLIP = 0.2


def _grpo_inputs(cpu, ref_lp, seed, old_noise=0.15):
    """pi_old log-probs = trainer + noise (kept off the clip boundaries); pi_vllm = the batch's."""
    g = np.random.default_rng(seed)
    mask = hp.npy(cpu["mask"]).astype(bool)
    old = ref_lp + old_noise * g.normal(size=ref_lp.shape)
    r = np.exp(ref_lp - old)
    near = (np.abs(r - (1 + CLIP)) < 1e-2) | (np.abs(r - (1 - CLIP)) < 1e-2)
    old[near] += 0.03
    old[~mask] = np.nan                                    # never read
    adv = orc.group_advantage(hp.npy(cpu["reward"]), hp.npy(cpu["group_id"]), cpu["P"], 1e-6)
    return old.astype(np.float32), adv.astype(np.float32)


def _run_gpu(dev, old, adv, accumulate=False, dW_init=None):
    prob = B.make_problem(dev)
    ws = B.alloc_workspace(prob, B.OAPL_FLAG_FUSED)
    N, S, d, V = dev["N"], dev["S"], dev["d"], dev["V"]
    nan = float("nan")
    out = dict(loss=torch.full((1,), nan, device="cuda"), seq_logp=torch.full((S,), nan, device="cuda"),
               token_logp=torch.full((N,), nan, device="cuda"), clip_frac=torch.full((1,), nan, device="cuda"),
               dH=torch.full((N, d), nan, dtype=torch.bfloat16, device="cuda"),
               dW=dW_init.clone() if dW_init is not None else torch.full((V, d), nan, device="cuda"))
    B.oapl_grpo_loss_fwd_bwd(prob, old, adv, CLIP, out["loss"], out["seq_logp"], out["token_logp"],
                             out["clip_frac"], out["dH"], out["dW"], accumulate, ws)
    out["status"] = B.oapl_get_last_status(ws)
    return out


def _check(cpu, seed=0):
    Hd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["H"]))
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["W"]))
    t, m, sid = hp.npy(cpu["targets"]), hp.npy(cpu["mask"]), hp.npy(cpu["seq_id"])
    ref_lp, _ = orc.token_logprobs(Hd, Wd, t, m)
    old, adv = _grpo_inputs(cpu, ref_lp, seed)
    q = hp.npy(cpu["logp_inf"])
    ref = orc.grpo_fwd(Hd, Wd, t, m, sid, np.where(m > 0, old, 0.0), np.where(m > 0, q, 0.0), adv, cpu["S"],
                       CLIP, cpu["loss_scale"])
    rdH, rdW = orc.token_coef_bwd(Hd, Wd, t, m, ref["coef"])
    dev = hp.to_dev(cpu)
    out = _run_gpu(dev, torch.from_numpy(old).cuda(), torch.from_numpy(adv).cuda())
    assert out["status"] == 0
    assert np.abs(hp.npy(out["token_logp"]) - ref["token_logp"]).max() <= hp.TOL_TOKEN
    assert np.all(np.abs(hp.npy(out["seq_logp"]) - ref["seq_logp"]) <= hp.TOL_REL * np.abs(ref["seq_logp"]) + 1e-6)
    live = m > 0
    wts = np.exp(np.where(live, old - q, 0.0)) * live
    scale = cpu["loss_scale"] * np.sum(wts * np.abs(adv[sid]) * ref["ratio"] / np.maximum(ref["T"][sid], 1))
    assert abs(float(out["loss"]) - ref["loss"]) <= hp.TOL_REL * scale + 1e-9
    assert float(out["clip_frac"]) == pytest.approx(ref["clip_frac"], abs=1e-6)
    dH = hp.npy(out["dH"].float()).astype(np.float64)
    assert np.all(dH[~live] == 0.0)
    assert np.all(dH[ref["clipped"]] == 0.0)             # clipped tokens carry no gradient at all
    assert hp.fro_rel(dH, rdH) <= hp.TOL_FRO
    assert hp.fro_rel(hp.npy(out["dW"]), rdW) <= hp.TOL_FRO
    return cpu, out, ref, (old, adv)


def test_group_advantage_entry_point():
    g = torch.Generator().manual_seed(5)
    S, P = 96, 7
    reward = torch.randn(S, generator=g)
    reward[:8] = 1.0
    group_id = torch.randint(1, P - 1, (S,), generator=g).to(torch.int32)
    group_id[:8] = 0                                        # a group with all-equal rewards
    for eps in (1e-6, 1.0):
        adv = torch.full((S,), 123.0, device="cuda")
        B.oapl_group_advantage(reward.cuda(), group_id.cuda(), P, eps, adv)
        want = orc.group_advantage(reward.numpy(), group_id.numpy(), P, eps)
        assert np.allclose(adv.cpu().numpy(), want, rtol=1e-5, atol=1e-6)
        assert float(adv[:8].abs().max()) == 0.0


def test_tiny_config():
    cpu, out, ref, _ = _check(synth.make_batch(synth.WORKLOADS["tiny"], seed=0))
    assert 0.02 < ref["clip_frac"] < 0.5                   # both branches are exercised


def test_ragged_shapes():
    wl = dataclasses.replace(synth.small_variant("14b-long", prompts=3, samples=3, live_rows=700),
                             d=320, V=1000 + 37)
    _check(synth.make_batch(wl, seed=2), seed=2)


@pytest.mark.parametrize("name,rows", [("1.5b", 600), ("7b", 450), ("lag-stress", 450)])
def test_small_variants_of_the_paper_shaped_configurations(name, rows):
    _check(synth.make_batch(synth.small_variant(name, prompts=2, samples=4, live_rows=rows), seed=0), seed=3)


def test_many_ranges_several_waves_and_accumulation(monkeypatch):
    monkeypatch.setenv("OAPL_STAGE_ROWS", "1024")
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                             padded_to=256, d=256, V=4096 + 72)
    cpu, out, ref, (old, adv) = _check(synth.make_batch(wl, seed=12), seed=4)
    dev = hp.to_dev(cpu)
    base = torch.randn(cpu["V"], cpu["d"], device="cuda")
    acc = _run_gpu(dev, torch.from_numpy(old).cuda(), torch.from_numpy(adv).cuda(), accumulate=True, dW_init=base)
    assert torch.allclose(acc["dW"], base + out["dW"], rtol=1e-6, atol=1e-7)
    again = _run_gpu(dev, torch.from_numpy(old).cuda(), torch.from_numpy(adv).cuda())
    for k in ("loss", "clip_frac", "token_logp", "dW"):     # bitwise reproducible
        assert torch.equal(again[k], out[k]), k


def test_degenerate_batches_and_argument_errors():
    cpu = synth.make_batch(synth.WORKLOADS["tiny"], seed=7)
    cpu["mask"][cpu["seq_id"] == 5] = 0                     # a rollout without response tokens
    cpu["live_tokens"] = int(cpu["mask"].sum())
    _check(cpu, seed=5)
    cpu["mask"][:] = 0                                      # nothing live: zero loss and gradients
    dev = hp.to_dev(cpu)
    z = torch.zeros(cpu["N"], device="cuda")
    out = _run_gpu(dev, z, torch.ones(cpu["S"], device="cuda"))
    assert out["status"] == 0 and float(out["loss"]) == 0.0 and float(out["clip_frac"]) == 0.0
    assert float(out["dH"].float().abs().max()) == 0.0 and float(out["dW"].abs().max()) == 0.0
    prob = B.make_problem(dev)
    ws = B.alloc_workspace(prob, B.OAPL_FLAG_FUSED)
    with pytest.raises(B.OaplError) as e:
        B.oapl_grpo_loss_fwd_bwd(prob, z, None, CLIP, out["loss"], None, None, None, out["dH"], out["dW"], False, ws)
    assert e.value.status == -1
    with pytest.raises(B.OaplError) as e:
        B.oapl_grpo_loss_fwd_bwd(prob, z, z, -0.5, out["loss"], None, None, None, out["dH"], out["dW"], False, ws)
    assert e.value.status == -1


def test_7b_full_size_sampled_rows():
    dev = synth.make_batch(synth.WORKLOADS["7b"], seed=0, device="cuda", beta=1.0)
    N, S, P = dev["N"], dev["S"], dev["P"]
    mask = dev["mask"].bool()
    g = torch.Generator(device="cuda").manual_seed(3)
    # pi_old: the engine's log-probs plus noise (the trainer's own are not known before the call)
    old = torch.where(mask, dev["logp_inf"] + 0.1 * torch.randn(N, device="cuda", generator=g),
                      torch.full_like(dev["logp_inf"], float("nan")))
    adv_np = orc.group_advantage(hp.npy(dev["reward"]), hp.npy(dev["group_id"]), P, 1e-6).astype(np.float32)
    out = _run_gpu(dev, old, torch.from_numpy(adv_np).cuda())
    assert out["status"] == 0
    # O(N) stages re-run by the oracle on the library's own token log-probs
    tok = hp.npy(out["token_logp"]).astype(np.float64)
    m, sid = hp.npy(dev["mask"]), hp.npy(dev["seq_id"])
    oldn, qn = hp.npy(old), hp.npy(dev["logp_inf"])
    ref = orc.grpo_from_logprobs(tok, np.where(m > 0, oldn, 0.0), np.where(m > 0, qn, 0.0), m, sid, adv_np, S,
                                 CLIP, dev["loss_scale"])
    scale = dev["loss_scale"] * np.sum(np.abs(adv_np[sid]) * (m > 0) / np.maximum(ref["T"][sid], 1))
    assert abs(float(out["loss"]) - ref["loss"]) <= 1e-4 * scale
    assert float(out["clip_frac"]) == pytest.approx(ref["clip_frac"], abs=1e-5)
    # dH of sampled rows from the oracle's coefficients of those rows
    live = torch.nonzero(mask).flatten()
    gg = torch.Generator().manual_seed(0)
    pick = torch.cat([torch.tensor([0, 255, 256, live.numel() - 1]), torch.randint(0, live.numel(), (28,), generator=gg)])
    rows = live[pick.to(live.device)]
    rn = hp.npy(rows)
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(dev["W"]))
    Hs = orc.bf16_bits_to_f64(synth.bf16_bits(dev["H"][rows]))
    want, _ = orc.token_coef_bwd(Hs, Wd, hp.npy(dev["targets"][rows]), np.ones(len(rn), dtype=np.uint8), ref["coef"][rn])
    got = hp.npy(out["dH"][rows].float()).astype(np.float64)
    assert hp.fro_rel(got, want) <= hp.TOL_FRO
    assert float(out["dH"][~mask].float().abs().max()) == 0.0
    col = out["dW"].double().sum(dim=0)                      # softmax rows sum to 1
    assert float(col.abs().max()) <= 1e-3 * float(out["dW"].double().abs().sum(dim=0).max())
    # sampled vocabulary rows of dW from the oracle's per-token coefficients
    vs = hp.sample_vocab_rows(dev, mask, 50, seed=4)
    assert vs.numel() >= 64
    want_w, = hp.oracle_vocab_rows_dW(dev, mask, tok, vs, [ref["coef"]], per_token=True)
    hp.assert_rows_close(hp.npy(out["dW"][vs.cuda()]).astype(np.float64), want_w, "grpo dW")

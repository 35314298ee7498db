"""Element-by-element parity of the CUDA path (through the C ABI) with the fp64 oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2602_19362_b200 import binding as B, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _check(wl, seed=0, fused=False, **kw):
    cpu = synth.make_batch(wl, seed=seed)
    out = hp.run_gpu(hp.to_dev(cpu), fused=fused, **kw)
    ref = hp.run_oracle(cpu, **kw)
    assert out["n_live"] == cpu["live_tokens"]
    hp.assert_parity(out, ref, hp.npy(cpu["mask"]))
    return cpu, out, ref


BOTH = pytest.mark.parametrize("fused", [False, True], ids=["two-calls", "single-call"])


@BOTH
def test_tiny_config(fused):
    _check(synth.WORKLOADS["tiny"], fused=fused)


@BOTH
def test_tiny_paper_temperatures_and_plain_sum(fused):
    # beta_v = 1, beta_loss = 1e-3 (the paper's hyper-parameter tables), Eq. 3's plain sum
    _check(synth.WORKLOADS["tiny"], seed=1, beta_v=1.0, beta_loss=1e-3, loss_scale=1.0, fused=fused)


@BOTH
def test_ragged_shapes(fused):
    # V not a multiple of the tile, d a multiple of 64 only, packed rows with masked prompt rows
    wl = dataclasses.replace(synth.small_variant("14b-long", prompts=3, samples=3, live_rows=700),
                             d=320, V=1000 + 37)
    _check(wl, seed=2, fused=fused)


def test_value_estimate_entry_point():
    from oracle import oapl_oracle as orc
    g = torch.Generator().manual_seed(5)
    S, P = 96, 7
    reward = torch.randn(S, generator=g)
    group_id = torch.randint(0, P - 1, (S,), generator=g).to(torch.int32)   # group P-1 is empty
    for beta in (1e-3, 0.1, 1.0, 10.0, 1e4):
        vhat = torch.full((P,), float("nan"), device="cuda")
        B.oapl_value_estimate(reward.cuda(), group_id.cuda(), P, beta, vhat)
        want = orc.value_estimate(reward.numpy(), group_id.numpy(), P, beta)
        assert np.allclose(vhat.cpu().numpy(), want, rtol=2e-6, atol=2e-6)
        assert vhat[P - 1].item() == 0.0


@BOTH
def test_many_chunks_and_waves_in_the_default_launch_configuration(fused):
    # about 20k response tokens: two default row chunks (18944 rows), several waves of row blocks
    # per chunk, sequences straddling tiles and chunks; small d and V keep the oracle fast
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                             padded_to=256, d=256, V=4096 + 72)
    cpu, out, ref = _check(wl, seed=11, fused=fused)
    assert cpu["live_tokens"] > 18944


def test_single_call_with_many_sequence_ranges(monkeypatch):
    # a staging capacity of 512 rows forces ~40 ranges of whole sequences (lengths up to 256)
    monkeypatch.setenv("OAPL_STAGE_ROWS", "512")
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                             padded_to=256, d=256, V=4096 + 72)
    _check(wl, seed=12, fused=True)


def test_single_call_reports_a_sequence_longer_than_the_staging_capacity(monkeypatch):
    monkeypatch.setenv("OAPL_STAGE_ROWS", "256")
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], length=("uniform", 300, 400), padded_to=512)
    cpu = synth.make_batch(wl, seed=13)
    out = hp.run_gpu(hp.to_dev(cpu), fused=True)
    assert out["status"] == -11


@BOTH
def test_batch_stats_entry_point(fused):
    from oracle import oapl_oracle as orc
    cpu = synth.make_batch(synth.WORKLOADS["tiny"], seed=14)
    cpu["mask"][cpu["seq_id"] == 3] = 0                  # a rollout without response tokens
    cpu["reward"][4:8] = 1.0                             # a group with all-equal rewards
    cpu["live_tokens"] = int(cpu["mask"].sum())
    dev = hp.to_dev(cpu)                                 # the problem struct points into these tensors
    out = hp.run_gpu(dev, fused=fused)
    ref = hp.run_oracle(cpu)
    hp.assert_parity(out, ref, hp.npy(cpu["mask"]))
    stats = torch.full((8,), float("nan"), device="cuda")
    B.oapl_batch_stats(out["prob"], out["vhat"], stats, out["ws"], B.OAPL_FLAG_FUSED if fused else 0)
    assert B.oapl_get_last_status(out["ws"]) == 0
    want = orc.batch_stats(ref["D"], ref["T"], hp.npy(cpu["reward"]), hp.npy(cpu["group_id"]), ref["vhat"], cpu["P"])
    got = dict(zip(B.STATS, hp.npy(stats)[:7].tolist()))
    assert got["live_tokens"] == want["live_tokens"] and got["frac_groups_all_equal"] == want["frac_groups_all_equal"]
    assert got["mean_reward"] == pytest.approx(want["mean_reward"], rel=1e-6)
    assert got["mean_advantage"] == pytest.approx(want["mean_advantage"], rel=1e-5, abs=1e-6)
    # the log-ratios inherit the error of the token log-probs: 5e-4 sqrt(T) per sequence (see helpers)
    tol = 5e-4 * np.sqrt(ref["T"].max() + 1)
    assert abs(got["mean_abs_log_ratio"] - want["mean_abs_log_ratio"]) <= tol
    assert abs(got["max_abs_log_ratio"] - want["max_abs_log_ratio"]) <= tol
    assert abs(got["mean_token_log_ratio"] - want["mean_token_log_ratio"]) <= hp.TOL_TOKEN
    assert float(stats[7]) == 0.0
    # without a loss forward on the workspace the call reports it
    prob = out["prob"]
    ws = B.alloc_workspace(prob, B.OAPL_FLAG_FUSED if fused else 0)
    tok = torch.zeros(cpu["N"], device="cuda")
    B.oapl_token_logprobs(prob, tok, None, ws)
    B.oapl_batch_stats(prob, out["vhat"], stats, ws, B.OAPL_FLAG_FUSED if fused else 0)
    assert B.oapl_get_last_status(ws) == -10

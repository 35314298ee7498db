"""Edge cases, error reporting and determinism of the CUDA path."""
import dataclasses

import numpy as np
import pytest
import torch

from paper_2602_19362_b200 import binding as B, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu
TINY = synth.WORKLOADS["tiny"]


@pytest.mark.parametrize("fused", [False, True], ids=["two-calls", "single-call"])
def test_bitwise_run_to_run_determinism(fused):
    dev = hp.to_dev(synth.make_batch(TINY, seed=3))
    a, b = hp.run_gpu(dev, fused=fused), hp.run_gpu(dev, fused=fused)
    for k in ("loss", "seq_logp", "vhat", "delta", "token_logp", "dW"):
        assert torch.equal(a[k], b[k]), k
    assert torch.equal(a["dH"].view(torch.int16), b["dH"].view(torch.int16))


def test_several_row_chunks_and_vocab_splits(monkeypatch):
    # 128-row chunks force many gradient chunks; dW must accumulate across them
    cpu = synth.make_batch(TINY, seed=4)
    ref = hp.run_oracle(cpu)
    for chunk, splits in (("128", "1"), ("256", "8"), ("384", "16")):
        monkeypatch.setenv("OAPL_CHUNK_ROWS", chunk)
        monkeypatch.setenv("OAPL_SPLITS", splits)
        out = hp.run_gpu(hp.to_dev(cpu))
        hp.assert_parity(out, ref, hp.npy(cpu["mask"]))


def test_accumulate_into_dW():
    cpu = synth.make_batch(TINY, seed=5)
    dev = hp.to_dev(cpu)
    base = torch.randn(cpu["V"], cpu["d"], device="cuda")
    plain = hp.run_gpu(dev)
    acc = hp.run_gpu(dev, accumulate=True, dW_init=base)
    assert torch.allclose(acc["dW"], base + plain["dW"], rtol=1e-6, atol=1e-7)


def test_token_logprobs_entry_point_and_null_outputs():
    cpu = synth.make_batch(TINY, seed=6)
    dev = hp.to_dev(cpu)
    ref = hp.run_oracle(cpu, backward=False)
    prob = B.make_problem({**dev, "group_id": None, "reward": None, "logp_inf": None})
    ws = B.alloc_workspace(prob)
    tok = torch.full((cpu["N"],), float("nan"), device="cuda")
    seq = torch.full((cpu["S"],), float("nan"), device="cuda")
    B.oapl_token_logprobs(prob, tok, seq, ws)
    assert B.oapl_get_last_status(ws) == 0
    assert np.abs(hp.npy(tok) - ref["token_logp"]).max() <= hp.TOL_TOKEN
    assert np.all(np.abs(hp.npy(seq) - ref["seq_logp"]) <= hp.TOL_REL * np.abs(ref["seq_logp"]))
    B.oapl_token_logprobs(prob, tok, None, ws)
    assert B.oapl_get_last_status(ws) == 0
    # a backward on a workspace whose last forward was not a loss forward is refused
    dH = torch.full((cpu["N"], cpu["d"]), 1.0, dtype=torch.bfloat16, device="cuda")
    dW = torch.full((cpu["V"], cpu["d"]), 1.0, device="cuda")
    full = B.make_problem(dev)
    B.oapl_loss_bwd(full, dH, dW, False, ws)
    assert B.oapl_get_last_status(ws) == -10


def test_degenerate_batches():
    cpu = synth.make_batch(TINY, seed=7)
    # (a) a sequence without any response token, scattered group membership, an empty group
    cpu["mask"][cpu["seq_id"] == 5] = 0
    cpu["group_id"] = torch.tensor([0, 2, 1, 2, 0, 1, 2, 0, 1, 2, 0, 1, 2, 1, 0, 2], dtype=torch.int32)
    cpu["live_tokens"] = int(cpu["mask"].sum())
    ref = hp.run_oracle(cpu)
    for fused in (False, True):
        out = hp.run_gpu(hp.to_dev(cpu), fused=fused)
        hp.assert_parity(out, ref, hp.npy(cpu["mask"]))
        assert float(out["seq_logp"][5]) == 0.0 and float(out["vhat"][3]) == 0.0
    # (b) nothing live at all: loss = lambda * sum A^2, gradients exactly zero
    cpu["mask"][:] = 0
    ref = hp.run_oracle(cpu)
    for fused in (False, True):
        out = hp.run_gpu(hp.to_dev(cpu), fused=fused)
        assert out["status"] == 0 and out["n_live"] == 0
        assert float(out["loss"]) == pytest.approx(ref["loss"], rel=1e-6)
        assert float(out["dH"].float().abs().max()) == 0.0 and float(out["dW"].abs().max()) == 0.0
    # (c) a single live row
    cpu["mask"][70] = 1
    cpu["targets"][70] = 17
    cpu["logp_inf"][70] = -8.0
    ref = hp.run_oracle(cpu)
    for fused in (False, True):
        hp.assert_parity(hp.run_gpu(hp.to_dev(cpu), fused=fused), ref, hp.npy(cpu["mask"]))


def test_one_token_vocab_and_all_equal_rewards():
    wl = dataclasses.replace(TINY, V=1, d=64)
    cpu = synth.make_batch(wl, seed=8)
    cpu["reward"][:] = 1.0                       # advantage 0 everywhere
    out = hp.run_gpu(hp.to_dev(cpu))
    ref = hp.run_oracle(cpu)
    assert out["status"] == 0
    assert float(out["token_logp"].abs().max()) <= 1e-5    # ln softmax over one token
    assert np.allclose(hp.npy(out["vhat"]), 1.0)
    assert float(out["loss"]) == pytest.approx(ref["loss"], rel=1e-3, abs=1e-6)
    assert float(out["dW"].abs().max()) < 1e-6


def test_device_detected_input_errors_are_reported_not_trapped():
    base = synth.make_batch(TINY, seed=9)
    bad = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in base.items()}
    first_live = int(torch.nonzero(bad["mask"])[0])
    bad["targets"][first_live] = bad["V"] + 5
    assert hp.run_gpu(hp.to_dev(bad))["status"] == -5
    bad = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in base.items()}
    bad["seq_id"][100] = 0                       # decreasing
    assert hp.run_gpu(hp.to_dev(bad))["status"] == -6
    bad = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in base.items()}
    bad["seq_id"][-1] = 99                       # outside [0,S)
    assert hp.run_gpu(hp.to_dev(bad))["status"] == -6
    bad = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in base.items()}
    bad["reward"][3] = float("inf")
    assert hp.run_gpu(hp.to_dev(bad))["status"] == -7
    bad = {k: (v.clone() if torch.is_tensor(v) else v) for k, v in base.items()}
    bad["group_id"][2] = 77
    assert hp.run_gpu(hp.to_dev(bad))["status"] == -7
    # the context is still usable afterwards
    good = hp.run_gpu(hp.to_dev(base))
    assert good["status"] == 0


def test_single_call_reports_a_target_far_below_the_largest_logit():
    # one row whose target logit is ~190 below the largest one: exp(z - z_target - 40) overflows
    # fp32; the single call must say so, the two-call path (online maximum) still matches the oracle
    wl = dataclasses.replace(TINY, d=64, V=512)
    cpu = synth.make_batch(wl, seed=10)
    row = int(torch.nonzero(cpu["mask"])[3])
    cpu["W"][5] = 0.0
    cpu["W"][5, 0] = 16.0
    cpu["W"][9] = 0.0
    cpu["W"][9, 0] = -8.0
    cpu["H"][row] = 0.0
    cpu["H"][row, 0] = 8.0                       # z[5] = 128, z[9] = -64, the others 0
    cpu["targets"][row] = 9
    cpu["logp_inf"][row] = -192.0
    assert hp.run_gpu(hp.to_dev(cpu), fused=True)["status"] == -12
    out = hp.run_gpu(hp.to_dev(cpu))
    ref = hp.run_oracle(cpu)
    assert out["status"] == 0
    assert abs(float(out["token_logp"][row]) - ref["token_logp"][row]) <= hp.TOL_TOKEN
    hp.assert_parity(out, ref, hp.npy(cpu["mask"]))


def test_two_streams_with_their_own_workspaces_give_the_single_stream_results():
    # Calls that overlap on the GPU compete for the SMs, so the CTA pairs of one launch may not all
    # be resident when they try to meet: the meetings must give up quietly and results must not change.
    wl = synth.small_variant("7b", prompts=2, samples=4, live_rows=450)
    devs = [hp.to_dev(synth.make_batch(wl, seed=s)) for s in (21, 22)]
    want = [hp.run_gpu(d, fused=True) for d in devs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    outs = [None, None]
    torch.cuda.synchronize()
    for rep in range(3):
        for i, (d, st) in enumerate(zip(devs, streams)):
            with torch.cuda.stream(st):
                outs[i] = hp.run_gpu_async(d)
        torch.cuda.synchronize()
    for o, w in zip(outs, want):
        assert B.oapl_get_last_status(o["ws"]) == 0
        for k in ("loss", "seq_logp", "token_logp", "dW"):
            assert torch.equal(o[k], w[k]), k
        assert torch.equal(o["dH"].view(torch.int16), w["dH"].view(torch.int16))


def test_nvtx_ranges_do_not_change_anything(monkeypatch):
    dev = hp.to_dev(synth.make_batch(TINY, seed=3))
    want = [hp.run_gpu(dev, fused=f) for f in (False, True)]
    monkeypatch.setenv("OAPL_NVTX", "1")
    for f, w in zip((False, True), want):
        got = hp.run_gpu(dev, fused=f)
        assert got["status"] == 0
        for k in ("loss", "seq_logp", "token_logp", "dW"):
            assert torch.equal(got[k], w[k]), k


@pytest.mark.parametrize("d,V", [(64, 7), (128, 255), (64, 256), (192, 257), (64, 511), (128, 512), (64, 513),
                                 (320, 1025), (64, 2049)])
def test_vocabulary_sizes_around_the_tile_boundaries(d, V):
    # 256 and 512 are the widths of one accumulator and of one sweep tile: sizes just below, at and
    # just above them, on both paths, with a handful of short sequences (one partial row block)
    wl = dataclasses.replace(TINY, prompts=2, samples=3, length=("uniform", 3, 40), padded_to=48, d=d, V=V)
    cpu = synth.make_batch(wl, seed=d + V)
    ref = hp.run_oracle(cpu)
    for fused in (False, True):
        hp.assert_parity(hp.run_gpu(hp.to_dev(cpu), fused=fused), ref, hp.npy(cpu["mask"]))


@pytest.mark.parametrize("rows", [1, 127, 128, 129, 257])
def test_row_counts_around_the_row_block(rows):
    # two rollouts of one prompt with `rows` response tokens each: the live rows end just below, at
    # and just above a 256-row block (2, 254, 256, 258, 514); unequal rewards keep the residual of
    # Eq. 3 away from a pure cancellation, so the loss tolerance means something
    wl = dataclasses.replace(TINY, prompts=1, samples=2, length=("uniform", rows, rows), padded_to=rows, d=128,
                             V=700)
    cpu = synth.make_batch(wl, seed=rows)
    cpu["reward"][:] = torch.tensor([1.0, 0.0])
    ref = hp.run_oracle(cpu)
    for fused in (False, True):
        out = hp.run_gpu(hp.to_dev(cpu), fused=fused)
        assert out["n_live"] == 2 * rows
        hp.assert_parity(out, ref, hp.npy(cpu["mask"]))

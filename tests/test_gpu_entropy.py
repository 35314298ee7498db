"""Policy-entropy statistic (oapl_entropy) against the fp64 oracle, through the C ABI.

Tolerance: H_n = lse_n - sum_v p z is formed from the same fp32 logits and fp32 sums as
the token log-probability, so it gets the same absolute bound (2e-3 nats); the means over
a sequence or the batch average such values and keep that bound."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu
TOL_ENT = 2e-3


def _oracle_entropy(cpu):
    Hd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["H"]))
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["W"]))
    ent = orc.token_entropy(Hd, Wd, hp.npy(cpu["mask"]))
    per_seq, mean = orc.sequence_entropy(ent, hp.npy(cpu["mask"]), hp.npy(cpu["seq_id"]), cpu["S"])
    return ent, per_seq, mean


def _gpu_entropy(dev, path):
    N, S = dev["N"], dev["S"]
    tok = torch.full((N,), float("nan"), device="cuda")
    seq = torch.full((S,), float("nan"), device="cuda")
    mean = torch.full((1,), float("nan"), device="cuda")
    if path == "token_logprobs":
        prob = B.make_problem({**dev, "group_id": None, "reward": None, "logp_inf": None})
        ws = B.alloc_workspace(prob)
        B.oapl_token_logprobs(prob, torch.empty(N, device="cuda"), None, ws)
        flags = 0
    else:
        out = hp.run_gpu(dev, fused=(path == "single-call"))
        prob, ws = out["prob"], out["ws"]
        flags = B.OAPL_FLAG_FUSED if path == "single-call" else 0
    B.oapl_entropy(prob, tok, seq, mean, ws, flags)
    assert B.oapl_get_last_status(ws) == 0
    return hp.npy(tok).astype(np.float64), hp.npy(seq).astype(np.float64), float(mean)


def _check(cpu, path):
    ent, per_seq, mean = _oracle_entropy(cpu)
    tok, seq, m = _gpu_entropy(hp.to_dev(cpu), path)
    mask = hp.npy(cpu["mask"])
    assert np.all(tok[mask == 0] == 0.0)
    assert np.abs(tok - ent).max() <= TOL_ENT
    assert np.abs(seq - per_seq).max() <= TOL_ENT
    assert abs(m - mean) <= TOL_ENT


PATHS = pytest.mark.parametrize("path", ["token_logprobs", "two-calls", "single-call"])


@PATHS
def test_tiny(path):
    _check(synth.make_batch(synth.WORKLOADS["tiny"], seed=0), path)


@PATHS
def test_ragged_shapes_and_several_waves(path):
    wl = dataclasses.replace(synth.small_variant("14b-long", prompts=3, samples=3, live_rows=700),
                             d=320, V=1000 + 37)
    _check(synth.make_batch(wl, seed=2), path)
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                             padded_to=256, d=256, V=4096 + 72)
    _check(synth.make_batch(wl, seed=11), path)


@pytest.mark.parametrize("name,rows", [("7b", 450), ("lag-stress", 450)])
def test_small_variants_of_the_paper_shaped_configurations(name, rows):
    # lag-stress scales the logits by 4: peaked distributions, entropies far below ln V
    cpu = synth.make_batch(synth.small_variant(name, prompts=2, samples=4, live_rows=rows), seed=0)
    for path in ("two-calls", "single-call"):
        _check(cpu, path)


def test_many_ranges_in_the_single_call_path(monkeypatch):
    monkeypatch.setenv("OAPL_STAGE_ROWS", "512")
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                             padded_to=256, d=256, V=4096 + 72)
    _check(synth.make_batch(wl, seed=12), "single-call")


def test_degenerate_batches_and_missing_forward():
    cpu = synth.make_batch(synth.WORKLOADS["tiny"], seed=7)
    cpu["mask"][cpu["seq_id"] == 5] = 0            # a sequence without response tokens
    cpu["live_tokens"] = int(cpu["mask"].sum())
    for path in ("two-calls", "single-call"):
        _check(cpu, path)
        _, seq, _ = _gpu_entropy(hp.to_dev(cpu), path)
        assert seq[5] == 0.0
    cpu["mask"][:] = 0                              # nothing live: all outputs 0
    for path in ("two-calls", "single-call"):
        tok, seq, m = _gpu_entropy(hp.to_dev(cpu), path)
        assert not tok.any() and not seq.any() and m == 0.0
    # a workspace no forward has written: reported, outputs untouched
    dev = hp.to_dev(synth.make_batch(synth.WORKLOADS["tiny"], seed=8))
    prob = B.make_problem(dev)
    ws = B.alloc_workspace(prob)
    ws.zero_()
    seq = torch.full((dev["S"],), -7.0, device="cuda")
    B.oapl_entropy(prob, None, seq, None, ws)
    assert B.oapl_get_last_status(ws) == -10
    assert bool((seq == -7.0).all())


def test_7b_full_size_sampled_rows():
    dev = synth.make_batch(synth.WORKLOADS["7b"], seed=0, device="cuda", beta=1.0)
    out = hp.run_gpu(dev, fused=True)
    N, S = dev["N"], dev["S"]
    tok = torch.full((N,), float("nan"), device="cuda")
    seq = torch.full((S,), float("nan"), device="cuda")
    mean = torch.full((1,), float("nan"), device="cuda")
    B.oapl_entropy(out["prob"], tok, seq, mean, out["ws"], B.OAPL_FLAG_FUSED)
    assert B.oapl_get_last_status(out["ws"]) == 0
    live = torch.nonzero(dev["mask"].bool()).flatten()
    g = torch.Generator().manual_seed(1)
    pick = torch.cat([torch.tensor([0, 255, 256, live.numel() - 1]), torch.randint(0, live.numel(), (28,), generator=g)])
    rows = live[pick.to(live.device)]
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(dev["W"]))
    Hs = orc.bf16_bits_to_f64(synth.bf16_bits(dev["H"][rows]))
    want = np.array([orc.row_entropy(Hs[i], Wd) for i in range(len(rows))])
    assert np.abs(hp.npy(tok[rows]) - want).max() <= TOL_ENT
    # the means re-derived by the oracle from the library's own per-token values (exact O(N) check)
    per_seq, m = orc.sequence_entropy(hp.npy(tok), hp.npy(dev["mask"]), hp.npy(dev["seq_id"]), S)
    assert np.allclose(hp.npy(seq), per_seq, rtol=1e-6, atol=1e-6)
    assert float(mean) == pytest.approx(m, rel=1e-6)
    assert float(tok[~dev["mask"].bool()].abs().max()) == 0.0

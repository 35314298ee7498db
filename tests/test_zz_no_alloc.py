"""oapl_token_logprobs_static: the workspace-free variant for callers that may not
allocate device memory at the call site (plug-ins under a foreign allocator, serving
loops with memory fixed at start-up).  Its scratch is one fixed array inside the library
that every call reuses, so the test runs two different problems back to back and checks
each against the ordinary entry point, which must give the same numbers.  Collected last
so that a failure here cannot hide the other tests behind `-x`."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu


def _both(wl, seed, oracle=False):
    cpu = synth.make_batch(wl, seed=seed)
    dev = hp.to_dev(cpu)
    prob = B.make_problem({**dev, "group_id": None, "reward": None, "logp_inf": None})
    N, S = cpu["N"], cpu["S"]
    ws = B.alloc_workspace(prob)
    tok_ref = torch.full((N,), float("nan"), device="cuda")
    seq_ref = torch.full((S,), float("nan"), device="cuda")
    B.oapl_token_logprobs(prob, tok_ref, seq_ref, ws)
    assert B.oapl_get_last_status(ws) == 0
    tok = torch.full((N,), float("nan"), device="cuda")
    seq = torch.full((S,), float("nan"), device="cuda")
    status = torch.full((1,), 123, dtype=torch.int32, device="cuda")
    B.oapl_token_logprobs_static(prob, tok, seq, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert torch.isfinite(tok).all() and torch.isfinite(seq).all()
    assert float((tok - tok_ref).abs().max()) <= hp.TOL_TOKEN
    assert torch.all((seq - seq_ref).abs() <= hp.TOL_REL * seq_ref.abs() + 1e-6)
    assert torch.all(tok[dev["mask"] == 0] == 0)
    if oracle:
        # and directly against the oracle on the same inputs, at the path's stated tolerances
        lp, _ = orc.token_logprobs(hp.f64(cpu["H"]), hp.f64(cpu["W"]), hp.npy(cpu["targets"]), hp.npy(cpu["mask"]))
        s_ref, _, _ = orc.sequence_sums(lp, np.zeros_like(lp), hp.npy(cpu["mask"]), hp.npy(cpu["seq_id"]), S)
        assert np.abs(hp.npy(tok) - lp).max() <= hp.TOL_TOKEN
        assert np.all(np.abs(hp.npy(seq) - s_ref) <= hp.TOL_REL * np.abs(s_ref) + 1e-6)


def test_static_scratch_matches_workspace_version_on_two_calls_in_a_row():
    big = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=4, samples=8, d=512, V=5000)   # N = 2048
    small = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=2, samples=2, d=128, V=333)  # N = 256
    _both(big, seed=21, oracle=True)
    _both(small, seed=22, oracle=True)      # reuses the array that still holds the larger problem's data
    _both(big, seed=23)


def test_static_scratch_at_the_limits_of_its_documented_sizes():
    # the widest hidden size with the most rows (the dense copy of H fills its 4 MB piece), then the
    # most sequences (2048 one-token sequences: the per-sequence pieces at their full size)
    widest = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=4, samples=8, d=1024, V=777)   # N = 2048
    _both(widest, seed=31, oracle=True)
    most_seqs = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=256, samples=8, length=("uniform", 1, 1),
                                    padded_to=1, d=64, V=300)                                    # S = N = 2048
    _both(most_seqs, seed=32, oracle=True)


def test_static_scratch_rejects_oversized_problems():
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=8, samples=8)                   # N = 4096
    dev = hp.to_dev(synth.make_batch(wl, seed=1))
    prob = B.make_problem({**dev, "group_id": None, "reward": None, "logp_inf": None})
    tok = torch.zeros(dev["N"], device="cuda")
    with pytest.raises(B.OaplError) as e:
        B.oapl_token_logprobs_static(prob, tok, None)
    assert e.value.status == -4

"""The seeded generators: shapes, determinism, structure of the paper-shaped batches."""
import numpy as np
import torch

from paper_2602_19362_b200 import synth


def test_tiny_batch_structure_and_determinism():
    wl = synth.WORKLOADS["tiny"]
    a = synth.make_batch(wl, seed=0)
    b = synth.make_batch(wl, seed=0)
    c = synth.make_batch(wl, seed=1)
    assert a["N"] == 16 * 64 and a["S"] == 16 and a["P"] == 4
    assert a["H"].dtype == torch.bfloat16 and a["H"].shape == (1024, 256)
    assert a["W"].shape == (4096, 256)
    for k in ("H", "W", "targets", "mask", "seq_id", "reward"):
        assert torch.equal(a[k], b[k]), k
    assert not torch.equal(a["H"], c["H"])
    assert int(a["mask"].sum()) == a["live_tokens"] == int(a["lengths"].sum())
    assert 16 <= int(a["lengths"].min()) and int(a["lengths"].max()) <= 64
    assert torch.all(a["seq_id"][1:] >= a["seq_id"][:-1])
    live = a["mask"].bool()
    assert torch.all((a["targets"][live] >= 0) & (a["targets"][live] < 4096))
    assert torch.all(a["targets"][~live] == -1)
    assert torch.isnan(a["logp_inf"][~live]).all() and torch.isfinite(a["logp_inf"][live]).all()
    assert set(a["reward"].tolist()) <= {0.0, 1.0}


def test_small_variants_keep_model_shape():
    for name in ("1.5b", "7b", "14b-long", "lag-stress"):
        wl = synth.small_variant(name, live_rows=600)
        full = synth.WORKLOADS[name]
        assert (wl.d, wl.V, wl.noise_std, wl.betas) == (full.d, full.V, full.noise_std, full.betas)
    wl = synth.small_variant("lag-stress", prompts=8, samples=4, live_rows=400)
    lens = synth._lengths(wl, 4000, torch.Generator().manual_seed(0))
    frac_clipped = float((lens == wl.length[4]).float().mean())
    assert 0.25 < frac_clipped < 0.35                      # 30 % of responses hit the cap


def test_sparse_rewards():
    wl = synth.WORKLOADS["lag-stress"]
    r = synth._rewards(wl, 4000, 16, torch.Generator().manual_seed(0)).reshape(4000, 16)
    assert abs(float(r.mean()) - 0.10) < 0.01
    assert abs(float((r.sum(1) == 0).float().mean()) - (0.25 + 0.75 * (1 - 0.1 / 0.75) ** 16)) < 0.03


def test_packed_layout_has_masked_prompt_rows():
    wl = synth.small_variant("14b-long", prompts=1, samples=2, live_rows=64)
    wl = synth.dataclasses.replace(wl, d=64, V=128)
    b = synth.make_batch(wl, seed=3)
    assert b["N"] == b["live_tokens"] + 3 * b["S"]
    assert b["mask"][:3].sum() == 0 and b["mask"][3] == 1
    assert np.array_equal(synth.bf16_bits(b["H"]).shape, (b["N"], 64))

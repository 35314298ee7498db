"""Parity on small variants of the paper-shaped configurations: same d, V, value
distributions, reward structure, noise level and temperatures as the full
configuration, but 2 prompts x 4 rollouts and a few hundred response tokens, which the
fp64 oracle finishes in seconds.  The rows still span several 128-row tiles with a
ragged tail and the vocabulary spans ~600 tiles with (for V = 151936) a half tile."""
import pytest

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,rows", [("1.5b", 600), ("7b", 450), ("14b-long", 400), ("lag-stress", 450)])
def test_small_variant_full_parity(name, rows):
    wl = synth.small_variant(name, prompts=2, samples=4, live_rows=rows)
    cpu = synth.make_batch(wl, seed=0)
    dev = hp.to_dev(cpu)
    betas = wl.betas
    out = hp.run_gpu(dev, beta_v=betas[0], beta_loss=betas[0])
    ref = hp.run_oracle(cpu, beta_v=betas[0], beta_loss=betas[0])
    mask = hp.npy(cpu["mask"])
    hp.assert_parity(out, ref, mask)
    # the single-call path (no recompute) on the same inputs
    hp.assert_parity(hp.run_gpu(dev, beta_v=betas[0], beta_loss=betas[0], fused=True), ref, mask)
    # remaining temperatures of the sweep, forward and backward on both paths: the oracle's forward
    # quantities only need its cached log-probs (Eq. 2 and Eq. 3 are O(S)), its gradient is
    # evaluated again with the new coefficients
    Hd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["H"]))
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["W"]))
    for b in betas[1:]:
        r = orc.loss_from_sums(ref["D"], hp.npy(cpu["reward"]), hp.npy(cpu["group_id"]), cpu["P"], b, b,
                               cpu["loss_scale"])
        r.update(token_logp=ref["token_logp"], seq_logp=ref["seq_logp"], T=ref["T"])
        r["dH"], r["dW"] = orc.loss_bwd(Hd, Wd, hp.npy(cpu["targets"]), mask, hp.npy(cpu["seq_id"]), r["coef"])
        hp.assert_parity(hp.run_gpu(dev, beta_v=b, beta_loss=b), r, mask)
        hp.assert_parity(hp.run_gpu(dev, beta_v=b, beta_loss=b, fused=True), r, mask)
    # the paper's own temperatures (beta_1 = 1 in Eq. 2, beta_2 = 1e-3 in Eq. 3)
    o = hp.run_gpu(dev, beta_v=1.0, beta_loss=1e-3, backward=False)
    r = orc.loss_from_sums(ref["D"], hp.npy(cpu["reward"]), hp.npy(cpu["group_id"]), cpu["P"], 1.0, 1e-3,
                           cpu["loss_scale"])
    r.update(token_logp=ref["token_logp"], seq_logp=ref["seq_logp"], T=ref["T"])
    hp.assert_parity(o, r, mask, backward=False)

"""The paper-shaped configurations at full size, in the launch configuration the benchmark
times, at every temperature the configuration sweeps.  The whole problem is out of reach for a
CPU (about 1e15 flops), so the oracle checks sampled outputs it can compute one by one --
at least 256 live rows and the two shortest whole sequences for the token log-probs, the
sampled rows of dH, at least 64 vocabulary rows of dW -- re-runs the O(N) stages on the
library's own token log-probs, and properties that hold at any size cover the rest."""
import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu

def invariants(dev, out, mask, fused):
    """Properties that hold at any size."""
    N = dev["N"]
    dH, dW = out["dH"], out["dW"]
    assert torch.isfinite(dW).all()
    for r0 in range(0, N, 65536):               # row blocks: no full-size fp32 copy of dH
        blk, dead = dH[r0:r0 + 65536], ~mask[r0:r0 + 65536]
        assert torch.isfinite(blk.float()).all()
        if bool(dead.any()):                    # packed layouts have no masked rows
            assert float(blk[dead].float().abs().max()) == 0.0               # masked rows exactly zero
    col = dW.double().sum(dim=0)                                             # softmax rows sum to 1
    assert float(col.abs().max()) <= 1e-3 * float(dW.double().abs().sum(dim=0).max())
    # <dH, H> = <dW, W> = sum_nv g[n,v] z[n,v].  Both sides use the same bf16 g, so what
    # separates them is the bf16 rounding of the dH output: independent relative errors of
    # at most 2^-9 per element, i.e. a standard deviation of about 2^-9/sqrt(3) * ||dH o H||_2
    # on the sum; allow six of those.
    lhs, sq = 0.0, 0.0
    for r0 in range(0, N, 65536):
        prod = dH[r0:r0 + 65536].double() * dev["H"][r0:r0 + 65536].double()
        lhs += float(prod.sum())
        sq += float((prod * prod).sum())
    rhs = float((dW.double() * dev["W"].double()).sum())
    sigma = 2.0 ** -9 / np.sqrt(3.0) * np.sqrt(sq)
    if fused:
        # the single call forms dW from bf16(scale_n * H[n, :]): a second, independent rounding of
        # the same size on the other side of the identity
        sigma *= np.sqrt(2.0)
    assert abs(lhs - rhs) <= 6.0 * sigma + 1e-4 * abs(rhs), (lhs, rhs, sigma)


@pytest.mark.parametrize("name,fused,betas", [("7b", True, (1.0, 0.5, 2.0)), ("7b", False, (1.0,)),
                                              ("1.5b", True, (1.0,)), ("14b-long", True, (1.0,)),
                                              ("lag-stress", True, (0.1, 10.0))],
                         ids=["7b-single-call", "7b-two-calls", "1.5b-single-call", "14b-long-single-call",
                              "lag-stress-single-call"])
def test_full_size_sampled_rows_and_invariants(name, fused, betas):
    # 1.5b: V = 151936 ends inside a 512-column tile; 14b-long: packed rows, sequences of up to 16384
    # tokens, d = 5120; lag-stress: 2.5 M response tokens, logits scaled by 4 (peaked distributions),
    # 25 % of the groups without any reward
    wl = synth.WORKLOADS[name]
    dev = synth.make_batch(wl, seed=0, device="cuda", beta=betas[0])
    N, S, P, d, V = (dev[k] for k in ("N", "S", "P", "d", "V"))
    mask = dev["mask"].bool()
    rows = hp.sample_rows(mask, 250, seed=0)
    assert rows.numel() >= 256
    vs = hp.sample_vocab_rows(dev, mask, 50, seed=2)
    assert vs.numel() >= 64

    # ---- the library, once per temperature; only what the checks need is kept
    kept = []
    for beta in betas:
        out = hp.run_gpu(dev, beta_v=beta, beta_loss=beta, fused=fused)
        assert out["status"] == 0 and out["n_live"] == dev["live_tokens"]
        out.pop("ws")                           # the largest configuration needs the room for the checks
        torch.cuda.empty_cache()
        invariants(dev, out, mask, fused)
        kept.append(dict(beta=beta, token_logp=out["token_logp"].clone(), seq_logp=hp.npy(out["seq_logp"]),
                         vhat=hp.npy(out["vhat"]), delta=hp.npy(out["delta"]), loss=float(out["loss"]),
                         dH_rows=hp.npy(out["dH"][rows].float()).astype(np.float64),
                         dW_rows=hp.npy(out["dW"][vs.cuda()]).astype(np.float64)))
        del out
        torch.cuda.empty_cache()
    for k in kept[1:]:                          # the token log-probs do not depend on the temperature
        assert torch.equal(k["token_logp"], kept[0]["token_logp"])
    tok = hp.npy(kept[0]["token_logp"]).astype(np.float64)

    # ---- sampled live rows and the two shortest whole sequences: token log-prob from the oracle
    Wd = hp.f64(dev["W"])
    lens = dev["lengths"]
    shortest = torch.argsort(lens)[:2]
    seq_rows = torch.nonzero(mask & torch.isin(dev["seq_id"], shortest.to(torch.int32).cuda())).flatten()
    all_rows = torch.cat([rows, seq_rows])
    lp_ref = np.concatenate([orc.token_logprobs(hp.f64(dev["H"][all_rows[c0:c0 + 1024]]), Wd,
                                                hp.npy(dev["targets"][all_rows[c0:c0 + 1024]]),
                                                np.ones(len(all_rows[c0:c0 + 1024]), dtype=np.uint8))[0]
                             for c0 in range(0, all_rows.numel(), 1024)])
    assert np.abs(tok[hp.npy(all_rows)] - lp_ref).max() <= hp.TOL_TOKEN
    # the shortest sequences' log-probabilities from the oracle's own token log-probs
    sid_rows = hp.npy(dev["seq_id"][seq_rows])
    for s in hp.npy(shortest):
        want_s = lp_ref[rows.numel():][sid_rows == s].sum()
        assert abs(kept[0]["seq_logp"][s] - want_s) <= hp.TOL_REL * abs(want_s)

    # ---- per temperature: the O(N) stages re-run by the oracle on the library's own token
    #      log-probs (exact check of the segmented sums, Eq. 2 and Eq. 3 at full size), then dH of
    #      the sampled rows from the oracle's coefficients of those rows' sequences
    s_ref, D, T = orc.sequence_sums(tok, hp.npy(dev["logp_inf"]), hp.npy(dev["mask"]), hp.npy(dev["seq_id"]), S)
    Hs = hp.f64(dev["H"][rows])
    tg = hp.npy(dev["targets"][rows])
    sid = hp.npy(dev["seq_id"][rows])
    coefs = []
    for k in kept:
        b = k["beta"]
        tail = orc.loss_from_sums(D, hp.npy(dev["reward"]), hp.npy(dev["group_id"]), P, b, b, dev["loss_scale"])
        assert np.allclose(k["seq_logp"], s_ref, rtol=1e-6)
        assert np.allclose(k["vhat"], tail["vhat"], rtol=1e-6, atol=1e-7)
        assert np.allclose(k["delta"], tail["delta"], rtol=1e-4, atol=1e-4)
        assert k["loss"] == pytest.approx(tail["loss"], rel=1e-5)
        coefs.append(tail["coef"])
        dH_ref, _ = orc.loss_bwd(Hs, Wd, tg, np.ones(len(sid), dtype=np.uint8), np.arange(len(sid)),
                                 tail["coef"][sid])
        hp.assert_rows_close(k["dH_rows"], dH_ref, ("dH", b))
    del Wd

    # ---- sampled vocabulary rows of dW, every temperature in one pass over the live rows
    for k, want in zip(kept, hp.oracle_vocab_rows_dW(dev, mask, tok, vs, coefs)):
        hp.assert_rows_close(k["dW_rows"], want, ("dW", k["beta"]))

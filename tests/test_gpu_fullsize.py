"""The 7B-scale configuration (and the two larger ones) at full size, in the launch
configuration the benchmark times.  The whole problem is out of reach for a CPU (about 1e15 flops), so the oracle
checks sampled outputs it can compute one by one, and properties that hold at any size
cover the rest."""
import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name,fused,beta", [("7b", True, 1.0), ("7b", False, 1.0), ("1.5b", True, 1.0),
                                             ("14b-long", True, 1.0), ("lag-stress", True, 0.1)],
                         ids=["7b-single-call", "7b-two-calls", "1.5b-single-call", "14b-long-single-call",
                              "lag-stress-single-call"])
def test_full_size_sampled_rows_and_invariants(name, fused, beta):
    # 1.5b: V = 151936 ends inside a 512-column tile; 14b-long: packed rows, sequences of up to 16384 tokens, d = 5120; lag-stress: 2.5 M response
    # tokens, logits scaled by 4 (peaked distributions), 25 % of the groups without any reward
    wl = synth.WORKLOADS[name]
    dev = synth.make_batch(wl, seed=0, device="cuda", beta=beta)
    out = hp.run_gpu(dev, fused=fused)
    assert out["status"] == 0 and out["n_live"] == dev["live_tokens"]
    N, S, P, d, V = (dev[k] for k in ("N", "S", "P", "d", "V"))
    mask = dev["mask"].bool()

    # --- sampled live rows (first, last, tile and chunk boundaries, random): token log-prob and dH row
    live = torch.nonzero(mask).flatten()
    g = torch.Generator().manual_seed(0)
    pick = torch.cat([torch.tensor([0, 1, 127, 128, 9471, 9472, 18943, 18944, live.numel() - 1]),
                      torch.randint(0, live.numel(), (41,), generator=g)])
    rows = live[pick.to(live.device)]
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(dev["W"]))
    Hs = orc.bf16_bits_to_f64(synth.bf16_bits(dev["H"][rows]))
    tg = hp.npy(dev["targets"][rows])
    lp_ref, _ = orc.token_logprobs(Hs, Wd, tg, np.ones(len(rows), dtype=np.uint8))
    assert np.abs(hp.npy(out["token_logp"][rows]) - lp_ref).max() <= hp.TOL_TOKEN

    # --- O(N) stages re-run by the oracle on the library's own token log-probs: exact check of
    #     the segmented sums, Eq. 2 and Eq. 3 at full size
    tok = hp.npy(out["token_logp"]).astype(np.float64)
    s, D, T = orc.sequence_sums(tok, hp.npy(dev["logp_inf"]), hp.npy(dev["mask"]), hp.npy(dev["seq_id"]), S)
    tail = orc.loss_from_sums(D, hp.npy(dev["reward"]), hp.npy(dev["group_id"]), P, beta, beta, dev["loss_scale"])
    assert np.allclose(hp.npy(out["seq_logp"]), s, rtol=1e-6)
    assert np.allclose(hp.npy(out["vhat"]), tail["vhat"], rtol=1e-6, atol=1e-7)
    assert np.allclose(hp.npy(out["delta"]), tail["delta"], rtol=1e-4, atol=1e-4)
    assert float(out["loss"]) == pytest.approx(tail["loss"], rel=1e-5)

    # --- dH of the sampled rows from the oracle's own coefficients of those rows' sequences
    coef = tail["coef"]
    sid = hp.npy(dev["seq_id"][rows])
    dH_ref, _ = orc.loss_bwd(Hs, Wd, tg, np.ones(len(rows), dtype=np.uint8), np.arange(len(rows)), coef[sid])
    got = hp.npy(out["dH"][rows].float()).astype(np.float64)
    assert hp.fro_rel(got, dH_ref) <= hp.TOL_FRO
    for i in range(len(rows)):
        assert hp.fro_rel(got[i], dH_ref[i]) <= 2 * hp.TOL_FRO

    # --- sampled vocabulary rows of dW (the most frequent targets, the first and last rows, random
    #     ones): z[n, v] of one vocabulary row costs O(N d), and the log-sum-exp of every live row
    #     follows from the (sample-checked) token log-probs as z[n, y_n] - lp_n
    if name == "7b" and fused:
        gv = torch.Generator().manual_seed(2)
        counts = torch.bincount(dev["targets"][mask].long(), minlength=V)
        vs = torch.cat([torch.topk(counts, 8).indices.cpu(), torch.tensor([0, 1, 255, 256, V - 1]),
                        torch.randint(0, V, (35,), generator=gv)]).unique()
        W_vs = orc.bf16_bits_to_f64(synth.bf16_bits(dev["W"][vs.cuda()]))
        live_idx = hp.npy(torch.nonzero(mask).flatten())
        want = np.zeros((len(vs), d))
        for c0 in range(0, len(live_idx), 32768):
            idx = live_idx[c0:c0 + 32768]
            it = torch.from_numpy(idx).cuda()
            Hc = orc.bf16_bits_to_f64(synth.bf16_bits(dev["H"][it]))
            tg_c = hp.npy(dev["targets"][it])
            Wt = orc.bf16_bits_to_f64(synth.bf16_bits(dev["W"][torch.from_numpy(tg_c).long().cuda()]))
            lse_c = np.einsum("nk,nk->n", Hc, Wt) - tok[idx]
            want += orc.vocab_rows_dW(hp.npy(vs), W_vs, Hc, tg_c, np.ones(len(idx), dtype=np.uint8),
                                      hp.npy(dev["seq_id"][it]), coef, lse_c)
        got_w = hp.npy(out["dW"][vs.cuda()]).astype(np.float64)
        assert hp.fro_rel(got_w, want) <= hp.TOL_FRO
        for i in range(len(vs)):
            assert hp.fro_rel(got_w[i], want[i]) <= 2 * hp.TOL_FRO, int(vs[i])

    # --- properties that hold at any size
    dH, dW = out["dH"], out["dW"]
    out.pop("ws")                               # the largest configuration needs the room for the checks
    torch.cuda.empty_cache()
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

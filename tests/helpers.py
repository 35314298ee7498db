"""Shared by the GPU parity tests: run the CUDA path through the C ABI and the
fp64 oracle on the same batch."""
import numpy as np
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B, synth

# tolerances stated for the path: per-token log-prob, sequence log-prob / loss, gradients
TOL_TOKEN = 2e-3
TOL_REL = 1e-3
TOL_FRO = 1e-2


def to_dev(batch):
    return {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in batch.items()}


def npy(t):
    return t.detach().cpu().numpy()


def f64(t):
    """A tensor of the batch as a float64 numpy array on the host (bf16 and fp32 widen exactly)."""
    return t.detach().cpu().to(torch.float64).numpy()


def run_gpu(dev, beta_v=None, beta_loss=None, loss_scale=None, backward=True, accumulate=False, dW_init=None,
            fused=False):
    """Run the CUDA path: oapl_loss_fwd (+ oapl_loss_bwd), or the single call
    oapl_loss_fwd_bwd when fused=True."""
    prob = B.make_problem(dev, beta_v, beta_loss, loss_scale)
    ws = B.alloc_workspace(prob, B.OAPL_FLAG_FUSED if fused else 0)
    N, S, P, d, V = (dev[k] for k in ("N", "S", "P", "d", "V"))
    out = dict(loss=torch.full((1,), float("nan"), device="cuda"),
               seq_logp=torch.full((S,), float("nan"), device="cuda"),
               vhat=torch.full((P,), float("nan"), device="cuda"),
               delta=torch.full((S,), float("nan"), device="cuda"),
               token_logp=torch.full((N,), float("nan"), device="cuda"))
    if backward:
        out["dH"] = torch.full((N, d), float("nan"), dtype=torch.bfloat16, device="cuda")
        out["dW"] = (dW_init.clone() if dW_init is not None
                     else torch.full((V, d), float("nan"), dtype=torch.float32, device="cuda"))
    if fused:
        assert backward
        B.oapl_loss_fwd_bwd(prob, out["loss"], out["seq_logp"], out["vhat"], out["delta"], out["token_logp"],
                            out["dH"], out["dW"], accumulate, ws)
    else:
        B.oapl_loss_fwd(prob, out["loss"], out["seq_logp"], out["vhat"], out["delta"], out["token_logp"], ws)
        if backward:
            B.oapl_loss_bwd(prob, out["dH"], out["dW"], accumulate, ws)
    out["status"] = B.oapl_get_last_status(ws)
    out["n_live"] = B.oapl_get_live_rows(ws)
    out["ws"] = ws
    out["prob"] = prob
    out["batch"] = dev          # the problem struct points into these tensors: keep them alive with it
    return out


def run_gpu_async(dev, fused=True):
    """Enqueue oapl_loss_fwd_bwd on the current stream without reading anything back (no
    synchronisation), so that calls on different streams can overlap on the GPU."""
    assert fused
    prob = B.make_problem(dev)
    ws = B.alloc_workspace(prob, B.OAPL_FLAG_FUSED)
    N, S, P, d, V = (dev[k] for k in ("N", "S", "P", "d", "V"))
    out = dict(loss=torch.zeros(1, device="cuda"), seq_logp=torch.zeros(S, device="cuda"),
               vhat=torch.zeros(P, device="cuda"), delta=torch.zeros(S, device="cuda"),
               token_logp=torch.zeros(N, device="cuda"),
               dH=torch.empty(N, d, dtype=torch.bfloat16, device="cuda"),
               dW=torch.empty(V, d, dtype=torch.float32, device="cuda"))
    B.oapl_loss_fwd_bwd(prob, out["loss"], out["seq_logp"], out["vhat"], out["delta"], out["token_logp"],
                        out["dH"], out["dW"], False, ws)
    out["ws"], out["prob"] = ws, prob
    return out


def run_oracle(cpu, beta_v=None, beta_loss=None, loss_scale=None, backward=True):
    Hd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["H"]))
    Wd = orc.bf16_bits_to_f64(synth.bf16_bits(cpu["W"]))
    bv = cpu["beta_v"] if beta_v is None else beta_v
    bl = cpu["beta_loss"] if beta_loss is None else beta_loss
    ls = cpu["loss_scale"] if loss_scale is None else loss_scale
    ref = orc.loss_fwd(Hd, Wd, npy(cpu["targets"]), npy(cpu["mask"]), npy(cpu["seq_id"]),
                       npy(cpu["group_id"]), npy(cpu["reward"]), npy(cpu["logp_inf"]),
                       cpu["S"], cpu["P"], bv, bl, ls)
    if backward:
        ref["dH"], ref["dW"] = orc.loss_bwd(Hd, Wd, npy(cpu["targets"]), npy(cpu["mask"]),
                                            npy(cpu["seq_id"]), ref["coef"])
    return ref


def fro_rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    den = np.linalg.norm(b)
    return np.linalg.norm(a - b) / den if den > 0 else np.linalg.norm(a - b)


def assert_parity(out, ref, mask, backward=True):
    assert out["status"] == 0, B.STATUS.get(out["status"], out["status"])
    tok = npy(out["token_logp"]).astype(np.float64)
    assert np.all(tok[mask == 0] == 0.0)
    assert np.abs(tok - ref["token_logp"]).max() <= TOL_TOKEN
    s = npy(out["seq_logp"]).astype(np.float64)
    assert np.all(np.abs(s - ref["seq_logp"]) <= TOL_REL * np.abs(ref["seq_logp"]) + 1e-6)
    assert np.allclose(npy(out["vhat"]), ref["vhat"], rtol=1e-5, atol=1e-6)
    # The residual delta_i = beta_2 D_i - A_i subtracts two O(1) numbers, so it is compared on the
    # scale of its parts (first term).  D_i sums T_i per-token differences lp - logp_inf, each with an
    # error of at most TOL_TOKEN = 2e-3 and no common sign.  Were those errors independent and spread
    # over the whole +-2e-3, the error of the sum would have a standard deviation of
    # 2e-3 sqrt(T_i / 3) = 1.15e-3 sqrt(T_i); the second term allows 5e-4 sqrt(T_i + 1), i.e. 0.43 of
    # that: it only passes when the per-token errors sit well inside their own bound.  It is not
    # scaled by beta_2, so for beta_2 < 1 it is looser than needed and the first term governs.
    scale = np.abs(ref["A"]) + np.abs(ref["delta"]) + 1e-3
    assert np.all(np.abs(npy(out["delta"]) - ref["delta"]) <= TOL_REL * scale + 5e-4 * np.sqrt(ref["T"] + 1))
    assert abs(float(out["loss"]) - ref["loss"]) <= TOL_REL * abs(ref["loss"]) + 1e-9
    if backward:
        dH = npy(out["dH"].float()).astype(np.float64)
        assert np.all(dH[mask == 0] == 0.0)
        assert np.isfinite(dH).all() and np.isfinite(npy(out["dW"])).all()
        assert fro_rel(dH, ref["dH"]) <= TOL_FRO
        assert fro_rel(npy(out["dW"]), ref["dW"]) <= TOL_FRO


# ---- sampling for the checks at full size ---------------------------------------------------
# rows of the compacted (live) row space at tile, chunk and range boundaries
BOUNDARY_ROWS = [0, 1, 127, 128, 255, 256, 9471, 9472, 18943, 18944, 32767, 32768, 65535, 65536]


def sample_rows(mask, n_random, seed):
    """Original row numbers of sampled live rows: boundaries of the compacted row space, the last
    live row, and random ones."""
    live = torch.nonzero(mask).flatten()
    g = torch.Generator().manual_seed(seed)
    pick = torch.cat([torch.tensor([r for r in BOUNDARY_ROWS if r < live.numel()] + [live.numel() - 1]),
                      torch.randint(0, live.numel(), (n_random,), generator=g)]).unique()
    return live[pick.to(live.device)]


def sample_vocab_rows(dev, mask, n_random, seed):
    """Vocabulary rows: the most frequent targets, the first and last rows, rows at the 256- and
    512-row tile boundaries, random ones."""
    V = dev["V"]
    counts = torch.bincount(dev["targets"][mask].long(), minlength=V)
    g = torch.Generator().manual_seed(seed)
    fixed = [0, 1, 255, 256, 511, 512, 513, V - 513, V - 257, V - 2, V - 1]
    return torch.cat([torch.topk(counts, 8).indices.cpu(), torch.tensor(fixed),
                      torch.randint(0, V, (n_random,), generator=g)]).unique()


def oracle_vocab_rows_dW(dev, mask, tok64, vs, coef_sets, per_token=False, chunk=32768):
    """Rows `vs` of dW from the oracle, for several coefficient sets at once (one pass over the
    live rows in chunks).  z[n, v] of one vocabulary row costs O(N d); the log-sum-exp of every
    live row follows from its (sample-checked) token log-prob as z[n, y_n] - lp_n.  coef_sets are
    per sequence, or per row (original row numbering) when per_token."""
    d = dev["d"]
    W_vs = f64(dev["W"][vs.cuda()])
    live_idx = torch.nonzero(mask).flatten()
    want = [np.zeros((len(vs), d)) for _ in coef_sets]
    for c0 in range(0, live_idx.numel(), chunk):
        it = live_idx[c0:c0 + chunk]
        idx = npy(it)
        Hc = f64(dev["H"][it])
        tg_c = npy(dev["targets"][it])
        Wt = f64(dev["W"][dev["targets"][it].long()])
        lse_c = np.einsum("nk,nk->n", Hc, Wt) - tok64[idx]
        ones = np.ones(len(idx), dtype=np.uint8)
        for k, coef in enumerate(coef_sets):
            if per_token:
                want[k] += orc.vocab_rows_dW(npy(vs), W_vs, Hc, tg_c, ones, np.arange(len(idx)), coef[idx], lse_c)
            else:
                want[k] += orc.vocab_rows_dW(npy(vs), W_vs, Hc, tg_c, ones, npy(dev["seq_id"][it]), coef,
                                             lse_c)
    return want


def assert_rows_close(got, want, what):
    assert fro_rel(got, want) <= TOL_FRO, what
    for i in range(len(want)):
        assert fro_rel(got[i], want[i]) <= 2 * TOL_FRO, (what, i)

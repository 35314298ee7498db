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
    # the residual subtracts two O(1) numbers; compare on the scale of its parts
    scale = np.abs(ref["A"]) + np.abs(ref["delta"]) + 1e-3
    assert np.all(np.abs(npy(out["delta"]) - ref["delta"]) <= TOL_REL * scale + 5e-4 * np.sqrt(ref["T"] + 1))
    assert abs(float(out["loss"]) - ref["loss"]) <= TOL_REL * abs(ref["loss"]) + 1e-9
    if backward:
        dH = npy(out["dH"].float()).astype(np.float64)
        assert np.all(dH[mask == 0] == 0.0)
        assert np.isfinite(dH).all() and np.isfinite(npy(out["dW"])).all()
        assert fro_rel(dH, ref["dH"]) <= TOL_FRO
        assert fro_rel(npy(out["dW"]), ref["dW"]) <= TOL_FRO

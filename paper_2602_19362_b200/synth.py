"""Seeded synthetic OAPL batches (inputs only).

This module builds the *data* a trainer step receives: hidden states, the
LM-head weight, sampled response tokens with the inference engine's
log-probabilities, rewards and the group structure.  It stands in for the
rollout buffer of Algorithm 1 (the paper's datasets, weights and inference
engine are not available), shaped like the paper's workloads: G = 8 or 16
rollouts per prompt, responses of up to 16384 tokens, Qwen-class hidden and
vocabulary sizes, binary rewards.

It contains none of the method's arithmetic (no Eq. 2, no Eq. 3, no gradient)
and is shared by the CPU oracle tests and the CUDA tests so that both sides
see byte-identical inputs.  The only model-like computation here is the
inference-engine stand-in: it samples each response token from
softmax(H . W^T) (Gumbel-max) and records that token's log-probability plus
Gaussian noise that emulates trainer/engine mismatch and policy lag.  It uses
plain torch ops in fp32 and is never used to check anything.
"""
from __future__ import annotations

import dataclasses
import math

import torch


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    d: int
    V: int
    prompts: int          # P
    samples: int          # G rollouts per prompt
    length: tuple         # ("uniform", lo, hi) | ("lognormal", median, sigma, lo, hi)
    padded_to: int        # 0 = packed rows; >0 = every sequence padded to this many rows
    h_rms_norm: bool      # scale each row of H to unit RMS (RMSNorm-like, unit gain)
    h_scale: float        # extra factor on H (exact in bf16 when a power of two)
    w_std: float          # W ~ N(0, w_std^2); 0 means 1/sqrt(d)
    targets: str          # "uniform" | "sampled"
    reward: tuple         # ("bernoulli", p) | ("sparse", p_one_overall, frac_groups_all_zero)
    noise_std: float      # per-token N(0, s^2) added to the engine's log-probs
    betas: tuple          # temperatures the paper-shaped config sweeps
    prompt_rows: int = 0  # packed layouts: masked prompt rows in front of each response


def _wl(**kw):
    return Workload(**kw)


WORKLOADS = {
    # the five paper-shaped configurations
    "tiny": _wl(name="tiny", d=256, V=4096, prompts=4, samples=4, length=("uniform", 16, 64),
                padded_to=64, h_rms_norm=False, h_scale=1.0, w_std=0.0, targets="uniform",
                reward=("bernoulli", 0.5), noise_std=0.05, betas=(1.0,)),
    "1.5b": _wl(name="1.5b", d=1536, V=151936, prompts=8, samples=8, length=("uniform", 256, 2048),
                padded_to=2048, h_rms_norm=True, h_scale=1.0, w_std=0.02, targets="sampled",
                reward=("bernoulli", 0.3), noise_std=0.1, betas=(1.0,)),
    "7b": _wl(name="7b", d=3584, V=152064, prompts=16, samples=8, length=("uniform", 512, 4096),
              padded_to=4096, h_rms_norm=True, h_scale=1.0, w_std=0.02, targets="sampled",
              reward=("bernoulli", 0.4), noise_std=0.2, betas=(0.5, 1.0, 2.0)),
    "14b-long": _wl(name="14b-long", d=5120, V=152064, prompts=4, samples=16,
                    length=("lognormal", 6000.0, 0.3, 1, 16384), padded_to=0, h_rms_norm=True,
                    h_scale=1.0, w_std=0.02, targets="sampled", reward=("bernoulli", 0.25),
                    noise_std=0.3, betas=(1.0,)),
    "lag-stress": _wl(name="lag-stress", d=4096, V=128256, prompts=32, samples=16,
                      length=("lognormal", 4849.0, 1.0, 1, 8192), padded_to=0, h_rms_norm=True,
                      h_scale=4.0, w_std=0.02, targets="sampled", reward=("sparse", 0.10, 0.25),
                      noise_std=1.0, betas=(0.1, 10.0)),
}


def small_variant(name: str, prompts: int = 2, samples: int = 4, live_rows: int = 1200) -> Workload:
    """Same d, V, distributions and betas as WORKLOADS[name], but few, short
    sequences (about `live_rows` response tokens in total) so that a CPU can
    evaluate the whole problem."""
    wl = WORKLOADS[name]
    S = prompts * samples
    mean = max(4, live_rows // S)
    if wl.length[0] == "uniform":
        lo, hi = wl.length[1], wl.length[2]
        ratio = lo / hi
        new_hi = max(2, int(round(2 * mean / (1 + ratio))))
        new_lo = max(1, int(round(new_hi * ratio)))
        length = ("uniform", new_lo, new_hi)
        padded = new_hi if wl.padded_to else 0
    else:
        _, med, sigma, lo, hi = wl.length
        scale = mean / med
        length = ("lognormal", med * scale, sigma, 1, max(2, int(round(hi * scale))))
        padded = 0
    return dataclasses.replace(wl, name=wl.name + "-S", prompts=prompts, samples=samples,
                               length=length, padded_to=padded,
                               prompt_rows=(3 if not wl.padded_to else 0))


def _lengths(wl: Workload, S: int, gen: torch.Generator) -> torch.Tensor:
    if wl.length[0] == "uniform":
        lo, hi = wl.length[1], wl.length[2]
        return torch.randint(lo, hi + 1, (S,), generator=gen, dtype=torch.int64)
    _, med, sigma, lo, hi = wl.length
    x = torch.exp(math.log(med) + sigma * torch.randn(S, generator=gen, dtype=torch.float64))
    return x.round().clamp(lo, hi).to(torch.int64)


def _rewards(wl: Workload, P: int, G: int, gen: torch.Generator) -> torch.Tensor:
    if wl.reward[0] == "bernoulli":
        return (torch.rand(P * G, generator=gen) < wl.reward[1]).to(torch.float32)
    _, p_one, frac_zero = wl.reward
    dead = torch.rand(P, generator=gen) < frac_zero
    p_live = p_one / (1.0 - frac_zero)
    r = (torch.rand(P, G, generator=gen) < p_live).to(torch.float32)
    r[dead] = 0.0
    return r.reshape(-1)


def engine_stand_in(H, W, mask, targets_mode, V, gen, row_chunk=2048):
    """Inference-engine stand-in: sample a token per live row from
    softmax(H . W^T) (or uniformly) and return (tokens int32, logp float32)."""
    N = H.shape[0]
    dev = H.device
    tokens = torch.zeros(N, dtype=torch.int32, device=dev)
    logp = torch.zeros(N, dtype=torch.float32, device=dev)
    live = torch.nonzero(mask, as_tuple=False).flatten()
    Wf = W.float()
    for c0 in range(0, live.numel(), row_chunk):
        idx = live[c0:c0 + row_chunk]
        z = H[idx].float() @ Wf.t()
        lsm = torch.log_softmax(z, dim=1)
        if targets_mode == "uniform":
            tok = torch.randint(0, V, (idx.numel(),), generator=gen, device=dev)
        else:
            u = torch.rand(z.shape, generator=gen, device=dev).clamp_(1e-20, 1.0)
            tok = torch.argmax(lsm - torch.log(-torch.log(u)), dim=1)
        tokens[idx] = tok.to(torch.int32)
        logp[idx] = lsm.gather(1, tok[:, None]).squeeze(1)
    return tokens, logp


def make_batch(wl: Workload, seed: int = 0, device: str = "cpu", beta: float | None = None) -> dict:
    """Build one batch.  Returns a dict of torch tensors on `device` plus the
    python scalars N, S, P, d, V, beta_v, beta_loss, loss_scale.

    Layout: rows of a sequence are contiguous; `seq_id` is non-decreasing.
    Padded workloads give every sequence `padded_to` rows with mask = 0 on the
    tail; packed workloads put `prompt_rows` masked rows before each response.
    Masked rows carry an out-of-range target (-1) and NaN in `logp_inf` to
    show that neither is read.
    """
    dev = torch.device(device)
    cpu_gen = torch.Generator(device="cpu").manual_seed(seed)
    gen = torch.Generator(device=dev).manual_seed(seed + 1)
    P, G = wl.prompts, wl.samples
    S = P * G
    lens = _lengths(wl, S, cpu_gen)
    reward = _rewards(wl, P, G, cpu_gen)
    group_id = torch.arange(S, dtype=torch.int32) // G

    if wl.padded_to:
        rows = torch.full((S,), wl.padded_to, dtype=torch.int64)
        lead = torch.zeros(S, dtype=torch.int64)
    else:
        lead = torch.full((S,), wl.prompt_rows, dtype=torch.int64)
        rows = lens + lead
    N = int(rows.sum())
    seq_id = torch.repeat_interleave(torch.arange(S, dtype=torch.int32), rows)
    start = torch.cumsum(rows, 0) - rows
    pos = torch.arange(N, dtype=torch.int64) - torch.repeat_interleave(start, rows)
    lead_r = torch.repeat_interleave(lead, rows)
    len_r = torch.repeat_interleave(lens, rows)
    mask = ((pos >= lead_r) & (pos < lead_r + len_r)).to(torch.uint8)

    seq_id, mask = seq_id.to(dev), mask.to(dev)
    d, V = wl.d, wl.V
    H = torch.empty(N, d, dtype=torch.bfloat16, device=dev)
    step = 65536
    for r0 in range(0, N, step):
        h = torch.randn(min(step, N - r0), d, generator=gen, device=dev, dtype=torch.float32)
        if wl.h_rms_norm:
            h = h * torch.rsqrt((h * h).mean(dim=1, keepdim=True))
        H[r0:r0 + step] = (h * wl.h_scale).to(torch.bfloat16)
    w_std = wl.w_std if wl.w_std > 0 else 1.0 / math.sqrt(d)
    W = torch.empty(V, d, dtype=torch.bfloat16, device=dev)
    for v0 in range(0, V, step):
        W[v0:v0 + step] = (w_std * torch.randn(min(step, V - v0), d, generator=gen, device=dev,
                                               dtype=torch.float32)).to(torch.bfloat16)

    tokens, logp = engine_stand_in(H, W, mask.bool(), wl.targets, V, gen)
    noise = wl.noise_std * torch.randn(N, generator=gen, device=dev, dtype=torch.float32)
    live = mask.bool()
    targets = torch.where(live, tokens, torch.full_like(tokens, -1))
    logp_inf = torch.where(live, logp + noise, torch.full_like(logp, float("nan")))

    b = wl.betas[0] if beta is None else beta
    return dict(name=wl.name, N=N, S=S, P=P, d=d, V=V, H=H, W=W, targets=targets, mask=mask,
                seq_id=seq_id, group_id=group_id.to(dev), reward=reward.to(dev),
                logp_inf=logp_inf, lengths=lens, beta_v=float(b), beta_loss=float(b),
                loss_scale=1.0 / S, live_tokens=int(lens.sum()))


def bf16_bits(t: torch.Tensor):
    """bfloat16 tensor -> numpy uint16 bit patterns (CPU)."""
    return t.detach().cpu().contiguous().view(torch.int16).numpy().view("uint16")

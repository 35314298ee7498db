"""AdamW step with gradient clipping by norm (oapl_adamw_step) against the fp64 oracle.

The kernels compute in fp32: m, v and the update are compared to 1e-5 relative (a handful of
fp32 roundings per element), the fp32 master weight additionally gets one fp32 rounding of
theta per step; the bf16 weight must be the exact round-to-nearest-even of the library's own
fp32 master value (integer work), and within one bf16 step of the oracle's."""
import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B

pytestmark = pytest.mark.gpu
MATH = dict(lr=1e-6, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=1e-2, clip_norm=1e-3)   # the paper's math table
CODE = dict(lr=1e-5, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=1e-2, clip_norm=1.0)   # code table (lr not printed)


def _run(n, hp, steps, with_master, seed, other=None, grad_scale=1e-3):
    # the C ABI takes the hyper-parameters as fp32: the oracle gets those same numbers
    # (1 - 0.999f differs from 0.001 by 1.3e-5 relative)
    hp = {k: float(np.float32(x)) for k, x in hp.items()}
    g = torch.Generator().manual_seed(seed)
    theta0 = (0.02 * torch.randn(n, generator=g)).to(torch.bfloat16)
    W = theta0.clone().cuda()
    master = theta0.float().cuda() if with_master else None
    m = torch.zeros(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    gn = torch.zeros(1, device="cuda")
    oth = None if other is None else torch.tensor([other], device="cuda")
    th_ref, m_ref, v_ref = theta0.double().numpy(), np.zeros(n), np.zeros(n)
    for step in range(1, steps + 1):
        grad = grad_scale * torch.randn(n, generator=g) * (1.0 if step != 2 else 1e-4)   # step 2 is not clipped
        B.oapl_adamw_step(W, master, grad.cuda(), m, v, step, hp["lr"], hp["beta1"], hp["beta2"], hp["eps"],
                          hp["weight_decay"], hp["clip_norm"], oth, gn)
        prev = th_ref
        if not with_master:
            prev = W_prev.double().numpy() if step > 1 else th_ref
        th_ref, m_ref, v_ref, norm = orc.adamw_step(prev, grad.double().numpy(), m_ref, v_ref, step,
                                                    other_sq_norm=0.0 if other is None else other, **hp)
        torch.cuda.synchronize()
        assert float(gn) == pytest.approx(norm, rel=1e-5)
        # beta1 m + (1-beta1) g can cancel: the absolute error scales with the terms, not the sum
        assert np.allclose(m.cpu().numpy(), m_ref, rtol=1e-5, atol=1e-6 * np.abs(m_ref).max())
        assert np.allclose(v.cpu().numpy(), v_ref, rtol=1e-5, atol=1e-20)
        upd = np.abs(th_ref - prev)
        if with_master:
            got = master.cpu().double().numpy()
            # each step rounds the fp32 master once (half an ulp, at most 2^-24 * 2 |theta|) and drops
            # the part of the decay below that; the oracle carries its own fp64 trajectory, so the
            # allowance grows with the step count
            assert np.all(np.abs(got - th_ref) <= 1e-5 * upd + step * 1.3e-7 * np.abs(th_ref))
            assert torch.equal(W.cpu(), master.cpu().to(torch.bfloat16))          # exact RN of the fp32 value
        want_bf16 = torch.from_numpy(th_ref).to(torch.bfloat16)
        ulp = torch.maximum(W.cpu().float().abs(), want_bf16.float().abs()) * 2.0 ** -7
        assert bool(((W.cpu().float() - want_bf16.float()).abs() <= ulp).all())
        W_prev = W.cpu().clone()
    return W, master, m, v


@pytest.mark.parametrize("n", [4096 * 256, 1000003, 5])
def test_master_weights_three_steps(n):
    _run(n, MATH, 3, True, seed=n % 97)


def test_bf16_parameter_without_master_and_other_parameters_norm():
    _run(300001, CODE, 3, False, seed=1, other=4.0, grad_scale=1.0)


def test_clipping_off_and_argument_errors():
    hp = dict(MATH, clip_norm=0.0)
    _run(70000, hp, 2, True, seed=2)
    W = torch.zeros(8, dtype=torch.bfloat16, device="cuda")
    f = torch.zeros(8, device="cuda")
    with pytest.raises(B.OaplError) as e:
        B.oapl_adamw_step(W, f, f, f, f, 0, 1e-3, 0.9, 0.95, 1e-8, 0.0, 1.0)      # step < 1
    assert e.value.status == -1
    with pytest.raises(B.OaplError) as e:
        B.oapl_adamw_step(W, f, f, f, f, 1, 1e-3, 1.0, 0.95, 1e-8, 0.0, 1.0)      # beta1 = 1
    assert e.value.status == -1
    with pytest.raises(B.OaplError) as e:
        B.oapl_adamw_step(W, f, f, f[1:], f, 1, 1e-3, 0.9, 0.95, 1e-8, 0.0, 1.0)  # misaligned m
    assert e.value.status == -2


def test_after_the_loss_gradient_at_the_tiny_configuration():
    # dW from the library's own backward feeds the optimizer step; the oracle repeats both
    from paper_2602_19362_b200 import synth
    from tests import helpers as hlp
    cpu = synth.make_batch(synth.WORKLOADS["tiny"], seed=0)
    dev = hlp.to_dev(cpu)
    out = hlp.run_gpu(dev, fused=True)
    ref = hlp.run_oracle(cpu)
    n = cpu["V"] * cpu["d"]
    W = dev["W"].clone().view(-1)
    master = W.float()
    m = torch.zeros(n, device="cuda")
    v = torch.zeros(n, device="cuda")
    B.oapl_adamw_step(W, master, out["dW"].view(-1), m, v, 1, 1e-3, 0.9, 0.95, 1e-8, 1e-2, 1e-3)
    th, _, _, _ = orc.adamw_step(cpu["W"].double().numpy().reshape(-1), ref["dW"].reshape(-1), np.zeros(n),
                                 np.zeros(n), 1, 1e-3, 0.9, 0.95, 1e-8, 1e-2, 1e-3)
    # first step: |update| = lr * |g| / (|g| + eps') ~ lr; gradients match to 1e-2, the update to that
    got = master.cpu().double().numpy()
    base = cpu["W"].double().numpy().reshape(-1)
    assert hlp.fro_rel(got - base, th - base) <= 2e-2

"""Bring-up check of the TMA/tcgen05 main loop in its four operand-major forms."""
import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B, synth

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("wide", [False, True], ids=["256x256", "256x512"])
@pytest.mark.parametrize("a_mn,b_mn", [(0, 0), (0, 1), (1, 1), (1, 0)])
# the last shape has 81 wide tiles for 74 CTA pairs: its partial second round is split into half-width tiles
@pytest.mark.parametrize("M,N,K", [(128, 256, 64), (384, 512, 320), (200, 264, 128), (1000, 1304, 1088),
                                   (520, 3000, 4096), (2304, 4608, 128)])
def test_debug_gemm(M, N, K, a_mn, b_mn, wide):
    g = torch.Generator().manual_seed(M * 7 + N * 3 + K + a_mn * 2 + b_mn)
    A = torch.randn(M, K, generator=g).to(torch.bfloat16)
    Bm = torch.randn(N, K, generator=g).to(torch.bfloat16)     # C = A . Bm^T
    ref = orc.logits(orc.bf16_bits_to_f64(synth.bf16_bits(A)), orc.bf16_bits_to_f64(synth.bf16_bits(Bm)))
    A_dev = (A.t().contiguous() if a_mn else A).cuda()
    B_dev = (Bm.t().contiguous() if b_mn else Bm).cuda()
    C = torch.full((M, N), float("nan"), device="cuda")
    err = torch.zeros(2, dtype=torch.int32, device="cuda")     # status word, lock-step counter
    B.oapl_debug_gemm(A_dev, B_dev, C, M, N, K, a_mn, b_mn, err, wide=wide)
    torch.cuda.synchronize()
    assert int(err[0].item()) == 0
    got = C.cpu().numpy().astype(np.float64)
    assert np.isfinite(got).all()
    assert np.abs(got - ref).max() <= 1e-3 * np.sqrt(K) + 1e-3 * np.abs(ref).max()

"""Same-GPU comparison of the library's tensor-core main loop with cuBLAS.

    python -m paper_2602_19362_b200.gemm_compare [--shapes 8192x8192x16384,32768x3584x152064] [--secs 3]

For every shape M x N x K it runs, back to back on the current GPU and each for `--secs`
seconds, torch.matmul (cuBLAS, bf16 in, bf16 out) and oapl_debug_gemm (the TMA/tcgen05 main
loop of every contraction of the library, fp32 out) with 256 x 512 and 256 x 256 tiles, while
nvidia-smi samples the SM clock.  One JSON line per run: TFLOP/s, median SM MHz, and the
fraction of the tensor rate that clock allows (4096 bf16 MACs per SM per cycle).  On a
power-capped GPU the clock differs between the runs, which is the point of the comparison.
A is stored [M, K], B is stored [K, N] (the layout of the dH contraction: B is MN-major).
"""
from __future__ import annotations

import argparse
import json
import time

import torch

from . import binding as B
from .clocks import ClockSampler


def _sustained(fn, flops, label, secs, sms):
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    t0, n = time.time(), 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    while time.time() - t0 < secs:
        for _ in range(3):
            fn()
        n += 3
        torch.cuda.synchronize()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    ck = sampler.stop()
    out = {"kernel": label, "ms": ms, "tflops": flops / ms / 1e9, "sm_mhz": ck["sm_mhz"], "reasons": ck["reasons"]}
    if ck["sm_mhz"]:
        out["frac_of_clock_rate"] = out["tflops"] / (sms * 4096 * 2 * ck["sm_mhz"] * 1e6 / 1e12)
    print(json.dumps(out), flush=True)
    time.sleep(1.0)


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--shapes", default="8192x8192x16384,32768x3584x152064")
    ap.add_argument("--secs", type=float, default=3.0)
    args = ap.parse_args()
    dev = torch.device("cuda", torch.cuda.current_device())
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    gen = torch.Generator(device=dev).manual_seed(0)
    err = torch.zeros(2, dtype=torch.int32, device=dev)
    for shape in args.shapes.split(","):
        M, N, K = (int(x) for x in shape.lower().split("x"))
        A = torch.empty(M, K, device=dev, dtype=torch.bfloat16)
        for r0 in range(0, M, 4096):
            A[r0:r0 + 4096] = torch.randn(min(4096, M - r0), K, device=dev, generator=gen).to(torch.bfloat16)
        Bt = torch.empty(K, N, device=dev, dtype=torch.bfloat16)
        for k0 in range(0, K, 16384):
            Bt[k0:k0 + 16384] = torch.randn(min(16384, K - k0), N, device=dev, generator=gen).to(torch.bfloat16)
        Cb = torch.empty(M, N, device=dev, dtype=torch.bfloat16)
        C32 = torch.empty(M, N, device=dev, dtype=torch.float32)
        flops = 2.0 * M * N * K
        print(json.dumps({"shape": [M, N, K]}), flush=True)
        _sustained(lambda: torch.matmul(A, Bt, out=Cb), flops, "cuBLAS (torch.matmul)", args.secs, sms)
        _sustained(lambda: B.oapl_debug_gemm(A, Bt, C32, M, N, K, 0, 1, err, wide=True), flops,
                   "oapl 256x512 tiles", args.secs, sms)
        _sustained(lambda: B.oapl_debug_gemm(A, Bt, C32, M, N, K, 0, 1, err, wide=False), flops,
                   "oapl 256x256 tiles", args.secs, sms)
        if int(err[0].item()) != 0:
            raise RuntimeError("oapl_debug_gemm reported a pipeline timeout")
        # a spot check of the last result against cuBLAS
        ref = torch.matmul(A[:256].float(), Bt[:, :256].float())
        diff = float((C32[:256, :256] - ref).abs().max())
        print(json.dumps({"max_abs_diff_256x256_corner": diff, "ref_abs_max": float(ref.abs().max())}), flush=True)
        del A, Bt, Cb, C32


if __name__ == "__main__":
    main()

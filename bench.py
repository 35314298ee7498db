#!/usr/bin/env python
"""Benchmark of the OAPL LM-head hot path (loss forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 7b] [--impl reference]

A step is one oapl_loss_fwd_bwd_ex call (Eq. 3 forward and gradient; `--path two-calls` times
oapl_loss_fwd + oapl_loss_bwd instead) over one synthetic batch shaped like the paper's
7B-scale trainer step (d=3584, V=152064, 16 prompts x 8 rollouts, response lengths
U[512,4096], padded layout).  The metric is response tokens per second; the roofline
object credits 6*N*d*V flops per step against the measured dense-bf16 peak.  Rank 0
prints one JSON line.

With --gpus N > 1 and no torchrun environment the script starts N ranks itself (one per GPU,
torch.distributed.run on 127.0.0.1); every rank holds its own prompts (weak scaling, W
replicated) and the step includes the NCCL all-reduce of dW, started on a second stream as
soon as dW is complete, under the last range's dH contraction.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "response tokens/sec for OAPL loss fwd+bwd"
UNIT = "tokens/s"
# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per live token of the single call's
# three contraction kinds: one ncu capture of one launch per kind on a reduced copy of the 7B
# workload that fills one range of whole sequences (--prompts 1 --samples 26 --seed 2: 64,704 live
# tokens, same d and V): logits 19.99 + 20.06 GB, dW 49.90 + 2.17 GB, dH 47.43 + 0.45 GB read +
# written.  The full workload is five such ranges and every kind's traffic grows in proportion to
# the ranges it processes, so a step's figure is this times its live tokens.
DRAM_BYTES_PER_TOKEN_7B = 140.00e9 / 64704


# ---------------------------------------------------------------------------- helpers
def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(burst=float(p["bf16_tflops"]), sustained=float(p["bf16_tflops_sustained"]),
                    hbm=float(p["hbm_gbs"]), source="measured")
    return dict(burst=1590.0, sustained=1400.0, hbm=6650.0, source="fallback")


from paper_2602_19362_b200.clocks import ClockSampler  # noqa: E402


def reduce_max(value: float, dist, device) -> float:
    """Max over ranks of a per-rank time (identity when not distributed)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def reduce_sum(value: float, dist, device) -> float:
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return value
    import torch
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


# ---------------------------------------------------------------------------- oracle arm
def oracle_sample(workload: str, live_rows: int):
    """A bounded sample of the workload for the CPU oracle: same d, V, distributions and
    betas, 2 prompts x 4 rollouts and about `live_rows` response tokens."""
    from oracle import oapl_oracle as orc
    from paper_2602_19362_b200 import synth
    wl = synth.small_variant(workload, prompts=2, samples=4, live_rows=live_rows) \
        if workload != "tiny" else synth.WORKLOADS["tiny"]
    b = synth.make_batch(wl, seed=0)
    npy = lambda t: t.numpy()
    args = dict(Hb=synth.bf16_bits(b["H"]), Wb=synth.bf16_bits(b["W"]), t=npy(b["targets"]),
                m=npy(b["mask"]), s=npy(b["seq_id"]), g=npy(b["group_id"]), r=npy(b["reward"]),
                q=npy(b["logp_inf"]))

    def step():
        Hd, Wd = orc.bf16_bits_to_f64(args["Hb"]), orc.bf16_bits_to_f64(args["Wb"])
        f = orc.loss_fwd(Hd, Wd, args["t"], args["m"], args["s"], args["g"], args["r"], args["q"],
                         b["S"], b["P"], b["beta_v"], b["beta_loss"], b["loss_scale"])
        orc.loss_bwd(Hd, Wd, args["t"], args["m"], args["s"], f["coef"])
        return f["loss"]

    desc = (f"{wl.name}: {b['live_tokens']} response tokens in {b['S']} sequences, d={wl.d}, V={wl.V}, "
            f"oracle loss fwd+bwd in fp64 numpy")
    return step, b["live_tokens"], desc


def host_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy  # noqa: F401  (loads BLAS before the thread count is read)
    step, tokens, desc = oracle_sample(args.workload, args.ref_rows)
    for _ in range(min(args.warmup, 1)):
        step()
    steps = max(1, min(args.steps, 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    dt = (time.perf_counter() - t0) / steps
    val = tokens / dt
    cores = host_threads()
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": args.workload, "sample": desc},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------- launcher
def free_port() -> int:
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        return sk.getsockname()[1]


def spawn_ranks(args) -> int:
    """Started as plain `python bench.py --gpus N` (no torchrun environment): run the same
    command line as N ranks under torch.distributed.run on this node and return its exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, cwd=ROOT)


def run_dry(args) -> None:
    """Launcher check without a GPU: the ranks meet over gloo, aggregate a made-up per-rank time and
    token count exactly as the timed arm does, and rank 0 prints a line marked as a dry run."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but {world} rank(s) came up")
    if world > 1:
        dist.init_process_group("gloo")
    ms = reduce_max(10.0 + rank, dist if world > 1 else None, torch.device("cpu"))
    tok = reduce_sum(1000.0, dist if world > 1 else None, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"dry_run": "launcher check only: no kernel ran, not a measurement", "metric": METRIC,
                          "value": 0.0, "unit": UNIT, "n_gpus": world, "steps": 0, "warmup": 0,
                          "ms_per_step": ms, "tokens_all_ranks": tok, "gpu_launches": 0}), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ---------------------------------------------------------------------------- CUDA arm
def run_cuda(args) -> None:
    import torch
    import torch.distributed as dist
    from paper_2602_19362_b200 import binding as B, dp, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but {world} rank(s) came up")
    if not torch.cuda.is_available() or torch.cuda.device_count() < world:
        raise SystemExit(f"{world} rank(s) need {world} CUDA device(s); {torch.cuda.device_count()} visible "
                         "(there is no CPU fallback)")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # cpu_baseline first (rank 0, N=1 only), before the device is busy
    cpu_base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        step, tokens, desc = oracle_sample(args.workload, args.ref_rows)
        t0 = time.perf_counter()
        step()
        dt = time.perf_counter() - t0
        cpu_base = {"value": tokens / dt, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                    "sample": desc, "seconds": dt}

    wl = synth.WORKLOADS[args.workload]
    if args.prompts or args.samples:      # reduced copies of the workload, for profiler captures
        import dataclasses
        wl = dataclasses.replace(wl, prompts=args.prompts or wl.prompts, samples=args.samples or wl.samples,
                                 name=wl.name + "-reduced")
    # data-parallel over prompts: every rank holds its own groups (weak scaling), W replicated
    batch = synth.make_batch(wl, seed=args.seed + rank, device=str(dev), beta=args.beta)
    N, S, P, d, V = (batch[k] for k in ("N", "S", "P", "d", "V"))
    n_live = batch["live_tokens"]
    # the loss normalises over the rollouts of all ranks
    prob = B.make_problem(batch, loss_scale=1.0 / (S * world))
    fused = args.path == "single-call"
    ws = B.alloc_workspace(prob, B.OAPL_FLAG_FUSED if fused else 0, device=dev)
    loss = torch.zeros(1, device=dev)
    seq_logp = torch.zeros(S, device=dev)
    vhat = torch.zeros(P, device=dev)
    delta = torch.zeros(S, device=dev)
    dH = torch.empty(N, d, dtype=torch.bfloat16, device=dev)
    dW = torch.empty(V, d, dtype=torch.float32, device=dev)

    grpo = args.objective == "grpo"
    if grpo:
        # the paper's baseline on the same pipeline: pi_old = the engine's log-probs plus noise,
        # group-normalised advantages, clip ratio 0.2
        if not fused:
            raise SystemExit("--objective grpo runs on the single-call path only")
        gen = torch.Generator(device=dev).manual_seed(args.seed + 1000 + rank)
        logp_old = batch["logp_inf"] + 0.1 * torch.randn(N, device=dev, generator=gen)
        adv = torch.zeros(S, device=dev)
        B.oapl_group_advantage(batch["reward"], batch["group_id"], P, 1e-6, adv)
        clip_frac = torch.zeros(1, device=dev)

    # what the host knows about the batch it built: the response-token count and the longest
    # response bound the number of range slots the single call enqueues
    comm_stream = torch.cuda.Stream() if world > 1 else None
    dW_ready = None
    if world > 1 and fused and not grpo:
        dW_ready = torch.cuda.Event()
        dW_ready.record()                      # torch creates the CUDA event at its first record
    opts = B.make_options(live_rows_bound=n_live, max_seq_rows_bound=int(batch["lengths"].max()),
                          dW_ready_event=dW_ready)

    def step(prob=prob, loss=loss, seq_logp=seq_logp, dH=dH, dW=dW):
        local_step(prob, loss, seq_logp, dH, dW)
        if world > 1:
            # the one exchange of the data-parallel step: sum of dW (and of the loss) over the ranks
            if dW_ready is not None:
                # dW is complete before the last range's dH contraction: NCCL runs under it
                handle = dp.start_allreduce_dW(dW, dW_ready, comm_stream)
                dp.finish_allreduce(handle, loss)
            else:
                dp.allreduce_outputs(loss, dW)

    def local_step(prob, loss, seq_logp, dH, dW):
        if grpo:
            B.oapl_grpo_loss_fwd_bwd(prob, logp_old, adv, 0.2, loss, seq_logp, None, clip_frac, dH, dW, False, ws)
        elif fused:
            B.oapl_loss_fwd_bwd_ex(prob, loss, seq_logp, vhat, delta, None, dH, dW, False, ws, opts)
        else:
            B.oapl_loss_fwd(prob, loss, seq_logp, vhat, delta, None, ws)
            B.oapl_loss_bwd(prob, dH, dW, False, ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    barrier()
    st = B.oapl_get_last_status(ws)
    if st != 0:
        raise RuntimeError(f"device status {B.STATUS.get(st, st)}")
    assert B.oapl_get_live_rows(ws) == n_live

    # ---- timed region: device-resident inputs
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    B.oapl_profile_enable(True)
    launches0 = B.oapl_launch_count()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
    barrier()
    ev[0].record()
    for k in range(args.steps):
        step()
        ev[k + 1].record()
    barrier()
    launches = B.oapl_launch_count() - launches0
    total_ms = ev[0].elapsed_time(ev[args.steps])
    step_ms = [ev[k].elapsed_time(ev[k + 1]) for k in range(args.steps)]
    prof, prof_dropped = B.oapl_profile_read(with_dropped=True)
    prof_mhz = B.oapl_profile_read_clocks()
    n_ranges = B.oapl_get_range_count(ws) if fused else None
    # the per-kind times are divided by the step count below: every step must have been recorded
    n_rec = sum(v[1] for v in prof.values())
    if prof_dropped or n_rec % args.steps:
        raise RuntimeError(f"contraction timing incomplete: {n_rec} launches recorded over {args.steps} steps, "
                           f"{prof_dropped} dropped")
    B.oapl_profile_enable(False)
    clocks = sampler.stop() if rank == 0 else None
    st = B.oapl_get_last_status(ws)
    if st != 0:
        raise RuntimeError(f"device status {B.STATUS.get(st, st)}")
    loss_val = float(loss.item())

    ms_step = reduce_max(total_ms / args.steps, dist if world > 1 else None, dev)
    tokens_all = reduce_sum(float(n_live), dist if world > 1 else None, dev)
    value = tokens_all / (ms_step * 1e-3)

    # ---- the optimizer step that follows (AdamW + clipping by norm on W), timed on its own:
    #      an HBM-bound kernel pair, 34 algorithmic bytes per element with an fp32 master copy
    adamw = None
    if rank == 0 and not args.no_adamw:
        n_el = V * d
        Wopt = batch["W"].clone().view(-1)
        master = Wopt.float()
        m_st, v_st = torch.zeros(n_el, device=dev), torch.zeros(n_el, device=dev)
        aws = None
        l0 = B.oapl_launch_count()
        times = []
        for it in range(1, 9):
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record()
            aws = B.oapl_adamw_step(Wopt, master, dW.view(-1), m_st, v_st, it, 1e-6, 0.9, 0.95, 1e-8, 1e-2, 1e-3,
                                    ws=aws)
            a1.record()
            torch.cuda.synchronize()
            times.append(a0.elapsed_time(a1))
        ms_a = statistics.median(times[3:])
        gbs = 34.0 * n_el / (ms_a * 1e-3) / 1e9
        hbm = measured_peaks()["hbm"]
        adamw = {"elements": n_el, "ms": ms_a, "launches_per_step": (B.oapl_launch_count() - l0) // 8,
                 "roofline": {"bound": "hbm", "achieved": gbs, "peak": hbm, "unit": "GB/s", "frac": gbs / hbm,
                              # DRAM bytes per element (33.8) measured by ncu on a 233 M-element weight,
                              # scaled by the element count
                              "traffic": 33.8 * n_el, "traffic_kind": "scaled from a reduced capture",
                              "bytes_per_element": 34,
                              "peak_kind": f"hbm_gbs of {measured_peaks()['source']}"}}
        del Wopt, master, m_st, v_st

    # ---- end to end: host-resident inputs and results, copies inside the timed region.
    # Every step copies its inputs from pinned host memory and its results (loss, sequence
    # log-probs, dH, dW) back.  The caller pipelines the steps the way a trainer would: two sets
    # of device buffers, one copy-in stream, the compute stream, one copy-out stream, so that the
    # copies of step k+1 and k-1 run under the kernels of step k.
    e2e = None
    if not args.no_e2e:
        names = ["H", "targets", "mask", "seq_id", "group_id", "reward", "logp_inf"]
        host_in = {k: batch[k].cpu().pin_memory() for k in names}
        host_out = {"loss": torch.empty(1).pin_memory(), "seq_logp": torch.empty(S).pin_memory(),
                    "dH": torch.empty(N, d, dtype=torch.bfloat16).pin_memory(),
                    "dW": torch.empty(V, d, dtype=torch.float32).pin_memory()}
        h2d = sum(t.numel() * t.element_size() for t in host_in.values())
        d2h = sum(t.numel() * t.element_size() for t in host_out.values())
        slots = []
        for i in range(2):
            b_i = batch if i == 0 else {k: (v.clone() if (torch.is_tensor(v) and k in names) else v)
                                        for k, v in batch.items()}
            o_i = {"loss": loss, "seq_logp": seq_logp, "dH": dH, "dW": dW} if i == 0 else \
                  {"loss": torch.zeros_like(loss), "seq_logp": torch.zeros_like(seq_logp),
                   "dH": torch.empty_like(dH), "dW": torch.empty_like(dW)}
            slots.append({"batch": b_i, "prob": B.make_problem(b_i, loss_scale=1.0 / (S * world)), "out": o_i,
                          "in_done": torch.cuda.Event(), "comp_done": torch.cuda.Event(),
                          "out_done": torch.cuda.Event()})
        s_in, s_out, s_comp = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()

        def e2e_steps(n):
            for k in range(n):
                sl = slots[k & 1]
                with torch.cuda.stream(s_in):
                    if k >= 2:
                        s_in.wait_event(sl["comp_done"])      # the step that read this input set is done
                    for name in names:
                        sl["batch"][name].copy_(host_in[name], non_blocking=True)
                    sl["in_done"].record(s_in)
                s_comp.wait_event(sl["in_done"])
                if k >= 2:
                    s_comp.wait_event(sl["out_done"])         # this output set has been copied out
                step(sl["prob"], sl["out"]["loss"], sl["out"]["seq_logp"], sl["out"]["dH"], sl["out"]["dW"])
                sl["comp_done"].record(s_comp)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(sl["comp_done"])
                    for name, t in host_out.items():
                        t.copy_(sl["out"][name], non_blocking=True)
                    sl["out_done"].record(s_out)
            for sl in slots[:min(n, 2)]:
                s_comp.wait_event(sl["out_done"])

        e2e_steps(2)
        barrier()
        n_e2e = max(10, args.steps)      # the first copy-in and the last copy-out of the loop are exposed: amortise them
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        e2e_steps(n_e2e)
        e1.record()
        barrier()
        e2e_ms = reduce_max(e0.elapsed_time(e1) / n_e2e, dist if world > 1 else None, dev)
        e2e = {"value": tokens_all / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms, "steps": n_e2e,
               "pipelining": "two device buffer sets; copy-in, compute and copy-out streams"}
        st = B.oapl_get_last_status(ws)
        if st != 0:
            raise RuntimeError(f"device status {B.STATUS.get(st, st)} in the end-to-end loop")
        del slots

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    flops_step = 6.0 * n_live * d * V          # credited: logits, dH, dW
    gemm_ms = sum(v[0] for v in prof.values()) / args.steps
    gemm_launches = sum(v[1] for v in prof.values()) // args.steps
    # dominant kernel = the tcgen05 contraction kernel (all its instantiations together).  The
    # single-call path executes 6*N*d*V flops per step; the two-call path recomputes the logits
    # in the backward and executes 8*N*d*V.
    exec_factor = 6.0 if fused else 8.0
    exec_tflops = exec_factor * n_live * d * V / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else None
    peak = peaks["sustained"]
    roofline = {"bound": "tensor", "kernel": "gemm_kernel (tcgen05, one template: " + ("lse_e|dW|dH)" if fused else "lse|grad|dH|dW)"),
                "executed_flops_per_step": exec_factor * n_live * d * V,
                "achieved": exec_tflops, "peak": peak, "unit": "TFLOP/s",
                "frac": exec_tflops / peak if exec_tflops else None,
                # DRAM bytes of the contraction launches of one step: the per-token figure of a reduced
                # capture times this step's live tokens; only for the workload and path it was taken on
                "traffic": (DRAM_BYTES_PER_TOKEN_7B * n_live
                            if (DRAM_BYTES_PER_TOKEN_7B and fused and not grpo and args.workload == "7b") else None),
                "traffic_kind": "scaled by live tokens from a reduced capture (one range of 64,704 tokens, same d and V)",
                "peak_kind": f"bf16_tflops_sustained of {peaks['source']}",
                "credited_tflops": flops_step / (ms_step * 1e-3) / 1e12,
                "credited_frac_of_sustained": flops_step / (ms_step * 1e-3) / 1e12 / peaks["sustained"],
                "credited_frac_of_burst": flops_step / (ms_step * 1e-3) / 1e12 / peaks["burst"],
                "credited_frac_of_nominal_2250": flops_step / (ms_step * 1e-3) / 1e12 / 2250.0,
                "contraction_ms_per_step": gemm_ms, "contraction_launches_per_step": gemm_launches,
                "by_kind_ms_per_step": {k: v[0] / args.steps for k, v in prof.items() if v[1]},
                "by_kind_sm_mhz": {k: round(prof_mhz[k]) for k, v in prof.items() if v[1]}}
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": f"{wl.name}-scale: d={d}, V={V}, {P} prompts x {wl.samples} rollouts, "
                                   f"lengths {wl.length}, padded_to={wl.padded_to}, beta={batch['beta_v']}",
                       "rows_N": N, "live_tokens_per_gpu": n_live, "parallelism": f"dp{world} over prompts" + (", NCCL all-reduce of dW and loss in the step" if world > 1 else ""),
                       "l2": "inputs larger than L2 (H, W, g chunk each > 126 MB); no flush needed",
                       "api": ("oapl_grpo_loss_fwd_bwd" if grpo else "oapl_loss_fwd_bwd_ex") if fused
                              else "oapl_loss_fwd + oapl_loss_bwd",
                       "host_bounds": None if (grpo or not fused) else
                       {"live_rows_bound": n_live, "max_seq_rows_bound": int(batch["lengths"].max())},
                       "ranges": n_ranges,
                       "exchange": None if world == 1 else
                       ("all-reduce of dW on a second stream behind the dW-ready event, under the last range's dH"
                        if dW_ready is not None else "all-reduce of dW and loss after the call"),
                       "objective": args.objective,
                       "step_ms": step_ms, "loss": loss_val},
            "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
            "gpu_launches_per_step": int(launches) // args.steps,
            "roofline": roofline, "cpu_baseline": cpu_base, "adamw_step": adamw}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="7b")
    ap.add_argument("--beta", type=float, default=1.0)
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--ref-rows", type=int, default=2048, help="response tokens in the CPU oracle sample")
    ap.add_argument("--prompts", type=int, default=0, help="override the number of prompts (profiling)")
    ap.add_argument("--samples", type=int, default=0, help="override rollouts per prompt (profiling)")
    ap.add_argument("--path", default="single-call", choices=["single-call", "two-calls"],
                    help="oapl_loss_fwd_bwd (no recompute) or oapl_loss_fwd + oapl_loss_bwd")
    ap.add_argument("--objective", default="oapl", choices=["oapl", "grpo"],
                    help="Eq. 3 (default, the headline metric) or the paper's GRPO baseline objective")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-adamw", action="store_true", help="skip the separately timed optimizer step")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--dry-run", action="store_true",
                    help="launcher check on CPU (gloo): start the ranks, aggregate, print; no kernel runs")
    args = ap.parse_args()
    if args.gpus < 1:
        raise SystemExit("--gpus must be >= 1")
    args.warmup = max(args.warmup, 3) if args.impl == "cuda" else args.warmup
    if args.impl == "reference":
        run_reference(args)        # the oracle on host cores: rank 0 alone, whatever N
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    if args.dry_run:
        run_dry(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()

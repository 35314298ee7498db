"""What a memory checker and a race detector would look for, checked through the C ABI:
every entry point stays inside the buffers it was given (patterned guard bands around the
workspace and every output), results are bit-for-bit reproducible at the sizes the benchmark
times (with and without the lock-step meetings of the CTA pairs), a pipeline wait that runs
out is reported as a status and leaves the context usable, and the call options of the
single call (host-side row bounds, the dW-ready event) behave as documented."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oapl_oracle as orc
from paper_2602_19362_b200 import binding as B, synth
from tests import helpers as hp

pytestmark = pytest.mark.gpu
GUARD = 4096
PATTERN = 0xA5


class Guarded:
    """`nbytes` of device memory at the given alignment with GUARD patterned bytes on both sides."""

    def __init__(self, nbytes, align=16):
        self.raw = torch.full((nbytes + 2 * GUARD + align,), PATTERN, dtype=torch.uint8, device="cuda")
        self.off = GUARD + (-(self.raw.data_ptr() + GUARD)) % align
        self.nbytes = nbytes
        self.bytes = self.raw[self.off:self.off + nbytes]

    def tensor(self, shape, dtype):
        return self.bytes.view(dtype).reshape(shape)

    def intact(self):
        lo, hi = self.raw[:self.off], self.raw[self.off + self.nbytes:]
        return bool((lo == PATTERN).all()) and bool((hi == PATTERN).all())


def guarded(shape, dtype, align=16):
    n = int(np.prod(shape)) * torch.empty(0, dtype=dtype).element_size()
    g = Guarded(n, align)
    return g, g.tensor(shape, dtype)


def test_no_entry_point_writes_outside_its_workspace_or_outputs():
    # odd sizes everywhere: V ends inside a tile, d is a multiple of 64 only, packed rows with masked
    # prompt rows, a row count that is not a multiple of anything
    wl = dataclasses.replace(synth.small_variant("14b-long", prompts=3, samples=3, live_rows=700), d=320, V=1037)
    cpu = synth.make_batch(wl, seed=2)
    dev = hp.to_dev(cpu)
    N, S, P, d, V = (cpu[k] for k in ("N", "S", "P", "d", "V"))
    prob = B.make_problem(dev)
    f32, bf16 = torch.float32, torch.bfloat16
    guards = []

    def out(shape, dtype):
        g, t = guarded(shape, dtype)
        guards.append(g)
        return t

    def workspace(flags):
        g = Guarded(B.oapl_workspace_bytes(prob, flags), align=1024)
        guards.append(g)
        return g.bytes

    def check(ws, what):
        assert B.oapl_get_last_status(ws) == 0, what
        torch.cuda.synchronize()
        for i, g in enumerate(guards):
            assert g.intact(), (what, i)

    # forward only, and its entropy read-back
    ws = workspace(0)
    tok, seq = out((N,), f32), out((S,), f32)
    B.oapl_token_logprobs(prob, tok, seq, ws)
    te, se, me = out((N,), f32), out((S,), f32), out((1,), f32)
    B.oapl_entropy(prob, te, se, me, ws)
    check(ws, "token_logprobs + entropy")
    # two calls
    loss, vhat, delta = out((1,), f32), out((P,), f32), out((S,), f32)
    dH, dW = out((N, d), bf16), out((V, d), f32)
    B.oapl_loss_fwd(prob, loss, seq, vhat, delta, tok, ws)
    B.oapl_loss_bwd(prob, dH, dW, False, ws)
    stats = out((8,), f32)
    B.oapl_batch_stats(prob, vhat, stats, ws)
    check(ws, "loss_fwd + loss_bwd + batch_stats")
    want_dW = dW.clone()
    # single call, plain and with options, and the GRPO objective on the same pipeline
    wsf = workspace(B.OAPL_FLAG_FUSED)
    B.oapl_loss_fwd_bwd(prob, loss, seq, vhat, delta, tok, dH, dW, False, wsf)
    check(wsf, "loss_fwd_bwd")
    assert hp.fro_rel(hp.npy(dW), hp.npy(want_dW)) <= hp.TOL_FRO
    ev = torch.cuda.Event()
    ev.record()
    opts = B.make_options(cpu["live_tokens"], int(cpu["lengths"].max()), ev)
    B.oapl_loss_fwd_bwd_ex(prob, loss, seq, vhat, delta, tok, dH, dW, False, wsf, opts)
    check(wsf, "loss_fwd_bwd_ex")
    adv, clip = out((S,), f32), out((1,), f32)
    B.oapl_group_advantage(dev["reward"], dev["group_id"], P, 1e-6, adv)
    old = torch.where(dev["mask"].bool(), dev["logp_inf"], torch.zeros_like(dev["logp_inf"]))
    B.oapl_grpo_loss_fwd_bwd(prob, old, adv, 0.2, loss, seq, tok, clip, dH, dW, False, wsf)
    check(wsf, "grpo_loss_fwd_bwd")
    # Eq. 2 alone, the optimizer step, the workspace-free forward
    B.oapl_value_estimate(dev["reward"], dev["group_id"], P, 0.7, vhat)
    n_el = V * d
    gW, Wb = guarded((n_el,), bf16)
    guards.append(gW)
    Wb.copy_(dev["W"].reshape(-1))
    master, m, v, gn = out((n_el,), f32), out((n_el,), f32), out((n_el,), f32), out((1,), f32)
    master.copy_(Wb.float())
    m.zero_()
    v.zero_()
    gws = Guarded(int(B.lib().oapl_adamw_workspace_bytes()), align=16)
    guards.append(gws)
    B.oapl_adamw_step(Wb, master, dW.reshape(-1), m, v, 1, 1e-3, 0.9, 0.95, 1e-8, 1e-2, 1.0, grad_norm=gn,
                      ws=gws.bytes)
    st = out((1,), torch.int32)
    B.oapl_token_logprobs_static(prob, tok, seq, st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    for i, g in enumerate(guards):
        assert g.intact(), ("value_estimate / adamw / static", i)


@pytest.mark.parametrize("name", ["1.5b", "7b"])
def test_full_size_single_call_is_bitwise_reproducible_with_and_without_the_meetings(name, monkeypatch):
    # at this size every mechanism whose timing varies from run to run is in play: the lock-step
    # meetings of the CTA pairs, several ranges of whole sequences with dW accumulated over them by
    # reduce-add, tail waves that are re-split; none of them may change a single bit
    dev = synth.make_batch(synth.WORKLOADS[name], seed=0, device="cuda")
    keys = ("loss", "seq_logp", "vhat", "delta", "token_logp", "dW")

    def run():
        o = hp.run_gpu(dev, fused=True)
        assert o["status"] == 0
        o.pop("ws")
        return o

    a = run()
    b = run()
    for k in keys:
        assert torch.equal(a[k], b[k]), k
    assert torch.equal(a["dH"].view(torch.int16), b["dH"].view(torch.int16))
    del b
    torch.cuda.empty_cache()
    monkeypatch.setenv("OAPL_SYNC_EVERY", "0")      # no meetings: the pairs drift apart freely
    c = run()
    for k in keys:
        assert torch.equal(a[k], c[k]), k
    assert torch.equal(a["dH"].view(torch.int16), c["dH"].view(torch.int16))


def test_a_pipeline_wait_that_runs_out_is_reported_and_the_context_stays_usable():
    # The load warps leave out one pipeline step, so the tensor-core warp's wait for it can never be
    # satisfied; with a limit of 2e6 cycles (about a millisecond) every role must give up, the
    # kernel must free its tensor memory and return, and the status word must say DEVICE_TIMEOUT.
    g = torch.Generator().manual_seed(1)
    M, N, K = 512, 1024, 1024
    A = torch.randn(M, K, generator=g).to(torch.bfloat16).cuda()
    Bm = torch.randn(N, K, generator=g).to(torch.bfloat16).cuda()
    ref = orc.logits(orc.bf16_bits_to_f64(synth.bf16_bits(A)), orc.bf16_bits_to_f64(synth.bf16_bits(Bm)))
    for wide in (True, False):
        C = torch.zeros(M, N, device="cuda")
        err = torch.zeros(2, dtype=torch.int32, device="cuda")
        B.oapl_debug_gemm(A, Bm, C, M, N, K, 0, 0, err, wide=wide, wait_cycles=2_000_000, skip_step=7)
        torch.cuda.synchronize()
        assert int(err[0].item()) == -8
        # the same context, the same kernel, no knob: the right product
        err.zero_()
        B.oapl_debug_gemm(A, Bm, C, M, N, K, 0, 0, err, wide=wide)
        torch.cuda.synchronize()
        assert int(err[0].item()) == 0
        got = C.cpu().numpy().astype(np.float64)
        assert np.abs(got - ref).max() <= 1e-3 * np.sqrt(K) + 1e-3 * np.abs(ref).max()
        # a short limit alone does not disturb a healthy launch
        err.zero_()
        B.oapl_debug_gemm(A, Bm, C, M, N, K, 0, 0, err, wide=wide, wait_cycles=50_000_000)
        torch.cuda.synchronize()
        assert int(err[0].item()) == 0
    # and the product path still runs
    cpu = synth.make_batch(synth.WORKLOADS["tiny"], seed=0)
    hp.assert_parity(hp.run_gpu(hp.to_dev(cpu), fused=True), hp.run_oracle(cpu), hp.npy(cpu["mask"]))


def test_call_options_bounds_event_and_range_count(monkeypatch):
    # 512-row staging forces about 40 ranges; with the exact bounds the call enqueues few empty
    # slots, results are those of the plain call bit for bit, and the event marks dW complete
    monkeypatch.setenv("OAPL_STAGE_ROWS", "512")
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                             padded_to=256, d=256, V=4096 + 72)
    cpu = synth.make_batch(wl, seed=12)
    dev = hp.to_dev(cpu)
    plain = hp.run_gpu(dev, fused=True)
    assert plain["status"] == 0
    n_ranges = B.oapl_get_range_count(plain["ws"])
    live, longest = cpu["live_tokens"], int(cpu["lengths"].max())
    slots = B.lib().oapl_range_slots(live, longest, 512, cpu["S"])
    assert 30 <= n_ranges <= slots <= B.lib().oapl_range_slots(cpu["N"], 0, 512, cpu["S"])

    prob, ws = plain["prob"], plain["ws"]
    N, S, P, d, V = (cpu[k] for k in ("N", "S", "P", "d", "V"))
    o = dict(loss=torch.zeros(1, device="cuda"), seq_logp=torch.zeros(S, device="cuda"),
             vhat=torch.zeros(P, device="cuda"), delta=torch.zeros(S, device="cuda"),
             token_logp=torch.zeros(N, device="cuda"), dH=torch.empty(N, d, dtype=torch.bfloat16, device="cuda"),
             dW=torch.empty(V, d, device="cuda"))
    ev = torch.cuda.Event()
    ev.record()
    side = torch.cuda.Stream()
    snap = torch.zeros_like(o["dW"])
    launches0 = B.oapl_launch_count()
    B.oapl_loss_fwd_bwd_ex(prob, o["loss"], o["seq_logp"], o["vhat"], o["delta"], o["token_logp"], o["dH"], o["dW"],
                           False, ws, B.make_options(live, longest, ev))
    launches_tight = B.oapl_launch_count() - launches0
    with torch.cuda.stream(side):
        side.wait_event(ev)                     # what a communication stream would do
        snap.copy_(o["dW"])
    torch.cuda.synchronize()
    assert B.oapl_get_last_status(ws) == 0 and B.oapl_get_range_count(ws) == n_ranges
    for k in ("loss", "seq_logp", "vhat", "delta", "token_logp", "dW"):
        assert torch.equal(o[k], plain[k]), k
    assert torch.equal(o["dH"].view(torch.int16), plain["dH"].view(torch.int16))
    assert torch.equal(snap, o["dW"])           # dW was already final when the event fired
    launches0 = B.oapl_launch_count()
    B.oapl_loss_fwd_bwd(prob, o["loss"], o["seq_logp"], o["vhat"], o["delta"], o["token_logp"], o["dH"], o["dW"],
                        False, ws)
    assert launches_tight < B.oapl_launch_count() - launches0
    # bounds that are too small are detected on the device
    B.oapl_loss_fwd_bwd_ex(prob, o["loss"], o["seq_logp"], o["vhat"], o["delta"], o["token_logp"], o["dH"], o["dW"],
                           False, ws, B.make_options(live // 4, longest, None))
    assert B.oapl_get_last_status(ws) == -13
    # and the next call on the same workspace is clean again
    B.oapl_loss_fwd_bwd_ex(prob, o["loss"], o["seq_logp"], o["vhat"], o["delta"], o["token_logp"], o["dH"], o["dW"],
                           False, ws, B.make_options(0, 0, None))
    assert B.oapl_get_last_status(ws) == 0
    assert torch.equal(o["dW"], plain["dW"])


def test_overlapped_exchange_plumbing_on_a_one_rank_nccl_group():
    # The data-parallel step: oapl_loss_fwd_bwd_ex records the dW-ready event, a second stream waits
    # for it and runs the NCCL all-reduce of dW while the compute stream finishes dH, then the loss
    # follows.  With one rank the sums are identities, so dW and the loss must come out bit for bit
    # as without the exchange; what is exercised is the event handle, the stream order and NCCL.
    import os
    import socket
    import torch.distributed as dist
    from paper_2602_19362_b200 import dp
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", torch.cuda.current_device()))
    try:
        wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=16, samples=8, length=("uniform", 64, 256),
                                 padded_to=256, d=256, V=4096 + 72)
        cpu = synth.make_batch(wl, seed=15)
        dev = hp.to_dev(cpu)
        plain = hp.run_gpu(dev, fused=True)
        prob, ws = plain["prob"], plain["ws"]
        N, S, P, d, V = (cpu[k] for k in ("N", "S", "P", "d", "V"))
        loss, seq = torch.zeros(1, device="cuda"), torch.zeros(S, device="cuda")
        vhat, delta = torch.zeros(P, device="cuda"), torch.zeros(S, device="cuda")
        dH = torch.empty(N, d, dtype=torch.bfloat16, device="cuda")
        dW = torch.empty(V, d, device="cuda")
        ev = torch.cuda.Event()
        ev.record()
        comm = torch.cuda.Stream()
        opts = B.make_options(cpu["live_tokens"], int(cpu["lengths"].max()), ev)
        for _ in range(3):                          # steps back to back, as in the timed loop
            B.oapl_loss_fwd_bwd_ex(prob, loss, seq, vhat, delta, None, dH, dW, False, ws, opts)
            handle = dp.start_allreduce_dW(dW, ev, comm)
            assert handle is not None
            dp.finish_allreduce(handle, loss)
        torch.cuda.synchronize()
        assert B.oapl_get_last_status(ws) == 0
        assert torch.equal(dW, plain["dW"]) and torch.equal(loss, plain["loss"])
        assert torch.equal(dH.view(torch.int16), plain["dH"].view(torch.int16))
    finally:
        dist.destroy_process_group()


def test_two_prompt_shards_run_one_after_the_other_sum_to_the_unsharded_step():
    # The data-parallel step on the CUDA path without a second GPU: the two ranks' shards (whole
    # groups, global loss_scale) are run one after the other on this GPU as independent calls, and
    # their dW and loss are added as the all-reduce would.  Against the unsharded call only the
    # summation order differs; against the oracle the stated tolerances hold.
    from paper_2602_19362_b200 import dp
    wl = dataclasses.replace(synth.WORKLOADS["tiny"], prompts=6, samples=4, length=("uniform", 20, 120),
                             padded_to=128, d=256, V=4096 + 72)
    cpu = synth.make_batch(wl, seed=17)
    ref = hp.run_oracle(cpu)
    whole = hp.run_gpu(hp.to_dev(cpu), fused=True)
    hp.assert_parity(whole, ref, hp.npy(cpu["mask"]))
    dW = torch.zeros_like(whole["dW"])
    loss = 0.0
    dH_rows, n_rows = [], 0
    for rank in range(2):
        shard = dp.shard_by_prompt(cpu, rank, 2)
        out = hp.run_gpu(hp.to_dev(shard), fused=True)
        assert out["status"] == 0 and out["n_live"] == shard["live_tokens"]
        dW += out["dW"]
        loss += float(out["loss"])
        dH_rows.append(out["dH"])
        n_rows += shard["N"]
    assert n_rows == cpu["N"]
    assert loss == pytest.approx(float(whole["loss"]), rel=1e-5)
    assert loss == pytest.approx(ref["loss"], rel=hp.TOL_REL)
    assert hp.fro_rel(hp.npy(dW), hp.npy(whole["dW"])) <= 1e-4
    assert hp.fro_rel(hp.npy(dW), ref["dW"]) <= hp.TOL_FRO
    dH = torch.cat(dH_rows).float()
    assert hp.fro_rel(hp.npy(dH), hp.npy(whole["dH"].float())) <= 2e-3      # bf16 outputs of slightly different sums
    assert hp.fro_rel(hp.npy(dH), ref["dH"]) <= hp.TOL_FRO

"""world_size-2 gloo check of the benchmark's cross-rank aggregation (max of the
per-rank times, sum of the per-rank token counts)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.reduce_max(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    tok = bench.reduce_sum(1000.0 * (rank + 1), dist, torch.device("cpu"))
    q.put((rank, ms, tok))
    dist.destroy_process_group()


def test_max_time_and_token_sum_over_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 3000.0), (1, 15.0, 3000.0)]


def test_identity_without_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_max(3.5, None, "cpu") == 3.5
    assert bench.reduce_sum(7.0, None, "cpu") == 7.0


def _dp_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import numpy as np
    from paper_2602_19362_b200 import dp, synth
    from tests import helpers_cpu as hc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    full = synth.make_batch(hc.DP_WORKLOAD, seed=3)
    shard = dp.shard_by_prompt(full, rank, world)
    ref = hc.oracle_step(shard)
    loss = torch.tensor([ref["loss"]], dtype=torch.float64)
    dW = torch.from_numpy(ref["dW"])
    dp.allreduce_outputs(loss, dW)
    q.put((rank, float(loss), dW.numpy(), shard["N"], shard["S"], shard["P"], ref["dH"], np.asarray(ref["vhat"])))
    dist.destroy_process_group()


def test_sharding_by_prompt_plus_allreduce_reproduces_the_single_rank_step():
    # Eq. 2 / Eq. 3 couple only rollouts of one prompt: two ranks holding whole groups, with the
    # global loss_scale, must sum to the one-rank loss and dW; dH rows stay with their rank
    import numpy as np
    from paper_2602_19362_b200 import dp, synth
    from tests import helpers_cpu as hc
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_dp_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=300) for _ in procs), key=lambda t: t[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    full = synth.make_batch(hc.DP_WORKLOAD, seed=3)
    ref = hc.oracle_step(full)
    for rank, loss, dW, N, S, P, dH, vhat in got:
        assert loss == pytest.approx(ref["loss"], rel=1e-12)
        assert np.allclose(dW, ref["dW"], rtol=1e-10, atol=1e-14)
    assert sum(g[3] for g in got) == full["N"] and sum(g[4] for g in got) == full["S"]
    assert sum(g[5] for g in got) == full["P"]
    assert np.allclose(np.concatenate([g[6] for g in got]), ref["dH"], rtol=1e-10, atol=1e-14)
    assert np.allclose(np.concatenate([g[7] for g in got]), ref["vhat"], rtol=1e-12)


def _overlap_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    from paper_2602_19362_b200 import dp, synth
    from tests import helpers_cpu as hc
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    full = synth.make_batch(hc.DP_WORKLOAD, seed=5)
    ref = hc.oracle_step(dp.shard_by_prompt(full, rank, world))
    # the exchange of the overlapped step: dW leaves as soon as it is complete, the rank goes on
    # (here: it only then forms its loss tensor, as the device finishes dH and the loss after dW),
    # and the scalar follows at the end
    dW_a = torch.from_numpy(ref["dW"].copy())
    handle = dp.start_allreduce_dW(dW_a)
    loss_a = torch.tensor([ref["loss"]], dtype=torch.float64)
    dp.finish_allreduce(handle, loss_a)
    # the plain exchange after the step
    dW_b, loss_b = torch.from_numpy(ref["dW"].copy()), torch.tensor([ref["loss"]], dtype=torch.float64)
    dp.allreduce_outputs(loss_b, dW_b)
    q.put((rank, bool(torch.equal(dW_a, dW_b)), float(loss_a), float(loss_b)))
    dist.destroy_process_group()


def test_exchange_started_when_dW_is_ready_equals_the_exchange_after_the_step():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_overlap_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=300) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert all(same for _, same, _, _ in got)
    assert got[0][2] == got[0][3] == got[1][2] == got[1][3]


def test_exchange_helpers_are_no_ops_without_a_process_group():
    from paper_2602_19362_b200 import dp
    dW, loss = torch.ones(4, 4), torch.ones(1)
    assert dp.start_allreduce_dW(dW) is None
    dp.finish_allreduce(None, loss)
    assert float(dW.sum()) == 16.0 and float(loss) == 1.0


def test_prompt_blocks_cover_every_prompt_once():
    from paper_2602_19362_b200 import dp
    for P, world in ((16, 8), (7, 3), (4, 4), (3, 5)):
        owned = [list(dp.prompts_of_rank(P, r, world)) for r in range(world)]
        assert sorted(sum(owned, [])) == list(range(P))
        assert max(map(len, owned)) - min(map(len, owned)) <= 1

"""Multi-rank host logic on CPU (gloo, world_size 2): replicas share weights, own their tokens,
and the reported time is the slowest rank's."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_05607_b200 import replicas, synth

CFG = synth.MoEConfig("mr", T=48, d=32, f=32, E=4, k=2, G=2, seed=5)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        t = replicas.make_rank_inputs(CFG, rank, "cpu")
        # weights identical on every rank, tokens differ
        sig = torch.tensor([t["w1"].float().sum().item(), t["w_gate"].sum().item(), t["x"].float().sum().item()],
                           dtype=torch.float64)
        gathered = [torch.zeros(3, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(gathered, sig)
        ms = replicas.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")     # rank 1 is the slow one
        dist.barrier()
        if rank == 0:
            out.put((torch.stack(gathered).tolist(), ms))
    finally:
        dist.destroy_process_group()


def test_replicas_share_weights_own_tokens_and_time_is_max():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    sigs, ms = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert sigs[0][0] == sigs[1][0] and sigs[0][1] == sigs[1][1]      # same weights, same gate
    assert sigs[0][2] != sigs[1][2]                                    # different tokens
    assert ms == 15.0                                                  # max over ranks
    assert replicas.whole_job_tokens_per_s(CFG, world, 10, ms) == CFG.T * 2 * 10 / 0.015


def test_single_process_helpers():
    assert replicas.rank_token_config(CFG, 0) is CFG
    assert replicas.rank_token_config(CFG, 3).seed == CFG.seed + 3 * replicas.TOKEN_SEED_STRIDE
    assert replicas.max_over_ranks(3.5, None, "cpu") == 3.5
    a = replicas.make_rank_inputs(CFG, 0, "cpu")
    b = replicas.make_rank_inputs(CFG, 1, "cpu")
    assert torch.equal(a["w2"], b["w2"]) and not torch.equal(a["x"], b["x"])

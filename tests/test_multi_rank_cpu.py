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


def _ep_exchange_worker(rank, world, port, out):
    """The exchange of the expert-parallel path with uneven, data-dependent split sizes: every rank sends
    rank-tagged rows, learns how many it will receive, receives them in sender order, and the return trip
    brings every row back to where it started."""
    from paper_2605_05607_b200 import ep
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        send_counts = [3 + rank, 1 + 2 * rank]                      # rows for rank 0, rank 1
        n = sum(send_counts)
        rows = (torch.arange(n * 4, dtype=torch.float32).reshape(n, 4) + 1000 * rank)
        recv_counts = ep.exchange_counts(send_counts)
        got = ep.all_to_all_rows(rows, send_counts, recv_counts)
        back = ep.all_to_all_rows(got * 2, recv_counts, send_counts)
        dist.barrier()
        out.put((rank, recv_counts, got.tolist(), bool(torch.equal(back, rows * 2))))
    finally:
        dist.destroy_process_group()


def test_ep_exchange_with_uneven_splits():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_ep_exchange_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = {}
    for _ in range(world):
        rank, recv_counts, got, round_trip = q.get(timeout=120)
        res[rank] = (recv_counts, got, round_trip)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    # rank 0 sends 3 rows to rank 0 and 1 to rank 1; rank 1 sends 4 to rank 0 and 3 to rank 1
    assert res[0][0] == [3, 4] and res[1][0] == [1, 3]
    r0 = torch.tensor(res[0][1])
    assert r0.shape == (7, 4) and r0[0, 0] == 0 and r0[3, 0] == 1000        # own rows first, then rank 1's first rows
    r1 = torch.tensor(res[1][1])
    assert r1.shape == (4, 4) and r1[0, 0] == 12 and r1[1, 0] == 1000 + 16   # rank 0's 4th row, then rank 1's rows 4..
    assert res[0][2] and res[1][2]                                           # the return trip restores the order


def test_bench_starts_its_own_ranks_and_reports_the_real_world_size():
    """`python bench.py --gpus 2` outside a launcher starts two ranks itself; n_gpus in the line is the real
    world size and the time is the slowest rank's (the stub step of rank r takes (1 + r) ms).  A launcher whose
    world size disagrees with --gpus is an error, not a silently mislabelled run."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--launcher-selftest", "--gpus", "2",
                          "--steps", "5"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = json.loads([ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1])
    assert line["n_gpus"] == 2 and line["steps"] == 5
    assert line["ms_per_step"] >= 2.0                                   # rank 1 is the slow one
    bad = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--launcher-selftest", "--gpus", "2",
                          "--steps", "1"], env=dict(env, WORLD_SIZE="1", RANK="0"), capture_output=True, text=True,
                         timeout=300)
    assert bad.returncode != 0 and "must agree" in bad.stderr


def _ep_wire_worker(rank, world, port, out):
    """Each rank routes its own tokens (uneven, skewed routing), builds the dispatch layout with the CPU oracle and
    derives its link traffic from the layout's counters; the totals are summed over the ranks."""
    import numpy as np
    from oracle import moe_oracle as O
    from paper_2605_05607_b200 import ep
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = synth.MoEConfig("epw", T=40 + 25 * rank, d=64, f=32, E=8, k=3, G=world, bias="zipf", zipf_s=1.3, seed=31 + rank)
        rng = np.random.default_rng(100 + rank)
        logits = rng.standard_normal((cfg.T, cfg.E)).astype(np.float32)
        idx, _ = O.route(logits, synth.make_bias(cfg).numpy(), cfg.k, cfg.score_fn)
        lay = O.layout(idx, cfg.E, cfg.G)
        st = ep.wire_stats(cfg, rank, lay["group_counts"], lay["expert_counts"])
        # brute force over every (token, slot): rows that leave this rank with and without the de-duplication
        dests = [{int(e) // cfg.m for e in row} - {rank} for row in idx]
        assert st["rows_dedup"] == sum(len(dd) for dd in dests)
        assert st["rows_point_to_point"] == sum(1 for row in idx for e in row if int(e) // cfg.m != rank)
        assert st["bytes_back_dedup"] == st["rows_dedup"] * 2 * cfg.d
        assert 0.0 <= st["bytes_removed_share"] < 1.0 and st["rows_dedup"] <= st["rows_point_to_point"]
        tot = torch.tensor([st["rows_dedup"], st["rows_point_to_point"]], dtype=torch.int64)
        dist.all_reduce(tot)
        dist.barrier()
        if rank == 0:
            out.put(tot.tolist())
    finally:
        dist.destroy_process_group()


def test_ep_wire_bytes_with_and_without_dedup_on_uneven_routing():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_ep_wire_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    dedup, p2p = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert 0 < dedup < p2p          # skewed top-3 over 2 groups of 4 experts: several experts of a token share a group

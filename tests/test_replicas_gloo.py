"""The N > 1 plumbing of the benchmark (independent replicas, barrier, max-over-ranks timing,
whole-job throughput) exercised with two CPU processes over gloo."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2511_03092_b200 import replicas, synth
    grp = replicas.init_from_env("gloo")
    assert (grp.rank, grp.world, grp.backend) == (rank, world, "gloo")
    # each replica draws its own sequences: seeds and therefore prompt lengths differ between ranks
    seed = grp.seed_for(2511)
    lengths = synth.draw_prompt_lengths(synth.CONFIGS[2], 4, seed)
    grp.barrier()
    elapsed_ms = 10.0 * (rank + 1)                     # rank 1 is the slow one
    tput, ms = grp.aggregate_throughput(units_this_rank=320.0, elapsed_ms_this_rank=elapsed_ms)
    out.put((rank, seed, lengths, tput, ms, grp.max_over_ranks(float(rank)), grp.is_root))
    grp.barrier()
    grp.close()


def test_two_replicas_aggregate_with_max_time_and_summed_work():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, l0, t0, ms0, mx0, root0), (r1, s1, l1, t1, ms1, mx1, root1) = res
    assert (r0, r1) == (0, 1) and root0 and not root1
    assert s0 != s1 and l0 != l1                       # disjoint synthetic sequences per replica
    assert ms0 == ms1 == 20.0                          # the slowest rank's time, on every rank
    assert abs(t0 - 640.0 / 0.020) < 1e-6 and t0 == t1  # all units / max time
    assert mx0 == mx1 == 1.0


def test_single_process_needs_no_process_group():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    from paper_2511_03092_b200 import replicas
    grp = replicas.init_from_env()
    assert grp.world == 1 and grp.backend is None and grp.is_root
    assert grp.max_over_ranks(3.5) == 3.5
    assert grp.aggregate_throughput(100.0, 50.0) == (2000.0, 50.0)
    grp.barrier(); grp.close()
    assert not torch.distributed.is_initialized()

"""The one exchange a multi-GPU deployment needs -- compressed caches from head-sharded compression
to sequence-sharded decode -- exercised with two and four CPU processes over gloo."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


N_SEQS, HKV, SC, D = 8, 4, 6, 16


def _full_cache(tag):
    """A cache whose every element encodes (tensor, sequence, head, row, dim), so that any misplacement shows."""
    t = torch.arange(N_SEQS * HKV * SC * D, dtype=torch.float32).view(N_SEQS, HKV, SC, D)
    return t + tag * 1e6


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2511_03092_b200 import handoff, replicas
    grp = replicas.init_from_env("gloo")
    heads = handoff.heads_of_rank(HKV, world, rank)
    k_loc = _full_cache(1)[:, heads.start:heads.stop].contiguous()      # what head-sharded compression leaves here
    v_loc = _full_cache(2)[:, heads.start:heads.stop].contiguous()
    seq_len = torch.arange(100, 100 + N_SEQS, dtype=torch.int32)
    valid = torch.arange(N_SEQS, dtype=torch.int32)
    k, v, sl, vt = handoff.handoff(k_loc, v_loc, seq_len, valid)
    k2, v2, _, _ = handoff.handoff(k_loc, None, seq_len, valid)         # latent layout: no V cache
    mine = handoff.sequences_of_rank(N_SEQS, world, rank)
    ok = (torch.equal(k, _full_cache(1)[mine.start:mine.stop]) and torch.equal(v, _full_cache(2)[mine.start:mine.stop])
          and torch.equal(k2, k) and v2 is None
          and sl.tolist() == list(range(100 + mine.start, 100 + mine.stop)) and vt.tolist() == list(mine))
    out.put((rank, bool(ok), tuple(k.shape)))
    grp.barrier()
    grp.close()


@pytest.mark.parametrize("world", [2, 4])
def test_handoff_gives_every_rank_all_heads_of_its_sequences(world):
    port = _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=180) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ok, shape in res:
        assert ok, f"rank {rank}: wrong cache after the hand-off"
        assert shape == (N_SEQS // world, HKV, SC, D)


def test_handoff_is_the_identity_on_one_rank():
    from paper_2511_03092_b200 import handoff
    k = _full_cache(1)
    seq_len = torch.arange(N_SEQS, dtype=torch.int32)
    k2, v2, sl, vt = handoff.handoff(k, None, seq_len, seq_len)
    assert k2 is k and v2 is None and torch.equal(sl, seq_len) and torch.equal(vt, seq_len)
    with pytest.raises(ValueError):
        handoff.heads_of_rank(6, 4, 0)

"""Hand-off of compressed caches from head-sharded compression to sequence-sharded decode.

Compression is independent per (sequence, KV head) and decode attention per (sequence, KV head)
as well, so several GPUs can shard either way with no exchange inside the path.  A deployment
that compresses with the KV heads spread over the ranks (each rank holds the prompts' K/V of
its own heads, as the paper's prefill does across sockets, Section 4.1) but decodes with whole
sequences per rank (Section 4.2) needs exactly one exchange in between: every rank sends, to
each other rank, its heads of the sequences that rank will decode.  This module is that
exchange -- one `all_to_all_single` per cache tensor over `torch.distributed` (NCCL on GPUs,
gloo on CPU) plus a local reordering; `seq_len` and `valid_topk` depend only on the prompt
length and are identical on every rank, so they are sliced, not exchanged.

No kernel of the library is involved, and single-GPU runs never come here.
"""
from __future__ import annotations

from typing import Optional, Tuple

import torch
import torch.distributed as dist


def heads_of_rank(n_kv_heads: int, world: int, rank: int) -> range:
    """KV heads compressed by `rank` (contiguous blocks; n_kv_heads must divide evenly)."""
    if n_kv_heads % world:
        raise ValueError(f"{n_kv_heads} KV heads do not divide over {world} ranks")
    per = n_kv_heads // world
    return range(rank * per, (rank + 1) * per)


def sequences_of_rank(n_seqs: int, world: int, rank: int) -> range:
    """Sequences decoded by `rank` (contiguous blocks; n_seqs must divide evenly)."""
    if n_seqs % world:
        raise ValueError(f"{n_seqs} sequences do not divide over {world} ranks")
    per = n_seqs // world
    return range(rank * per, (rank + 1) * per)


def exchange_cache(cache_heads: torch.Tensor, group=None) -> torch.Tensor:
    """cache_heads: [n_seqs][heads_local][Sc][d] -- this rank's heads of every sequence's compressed
    cache.  Returns [n_seqs / world][heads_local * world][Sc][d]: every head of this rank's sequences,
    heads in global order.  With one rank the input is returned unchanged."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    if world == 1:
        return cache_heads
    n_seqs, h_loc, sc, d = cache_heads.shape
    if n_seqs % world:
        raise ValueError(f"{n_seqs} sequences do not divide over {world} ranks")
    per = n_seqs // world
    send = cache_heads.contiguous()                      # block r of `per` sequences goes to rank r
    recv = torch.empty_like(send)                        # block r: rank r's heads of my sequences
    dist.all_to_all_single(recv, send, group=group)
    # [src rank][seq][head][Sc][d] -> [seq][src rank][head][Sc][d] -> heads in global order
    return recv.view(world, per, h_loc, sc, d).permute(1, 0, 2, 3, 4).reshape(per, world * h_loc, sc, d).contiguous()


def handoff(k_cache_heads: torch.Tensor, v_cache_heads: Optional[torch.Tensor], seq_len: torch.Tensor,
            valid_topk: torch.Tensor, group=None) -> Tuple[torch.Tensor, Optional[torch.Tensor], torch.Tensor, torch.Tensor]:
    """Caches as written by head-sharded `snap_compress` calls (max_seqs = all sequences, n_kv_heads =
    this rank's share) -> caches for sequence-sharded `snap_decode_attn` calls (max_seqs = this rank's
    sequences, all KV heads), with this rank's slice of the per-sequence state."""
    world = dist.get_world_size(group) if dist.is_initialized() else 1
    rank = dist.get_rank(group) if dist.is_initialized() else 0
    k = exchange_cache(k_cache_heads, group)
    v = None if v_cache_heads is None else exchange_cache(v_cache_heads, group)
    mine = sequences_of_rank(seq_len.shape[0], world, rank)
    return k, v, seq_len[mine.start:mine.stop].clone(), valid_topk[mine.start:mine.stop].clone()

"""Token-range sharding of one decode-attention problem over several GPUs.

The CPU/GPU split of Section 4.2 (one device takes the older tokens, the other the recent ones, and the
softmax is taken over their union) generalises to N devices: rank r holds the pages of its own token
range, runs ``hg_attn_decode`` on it, and the ranks exchange one merged row per (sequence, query head).
A merged row ``(out, lse)`` is itself a softmax partial, ``(o, m, l) = (out, lse, 1)``, because
``e^{lse} * out`` is the un-normalised weighted sum of the rank's tokens and ``e^{lse}`` its weight;
so the exchange is one all-gather of ``B * Hq * (D + 1)`` floats per rank and the combine is the
library's own ``hg_attn_merge`` over ``world_size`` sources.  Remote rows are landed in this rank's own
buffer by the collective before any kernel reads them.

This module holds the host-side plan (which rank takes which tokens), the packing of the exchanged
record and the calls; the arithmetic stays in the CUDA library.
"""
from __future__ import annotations

from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist

from . import binding as hg

RECORD_ALIGN = 64      # floats; keeps every rank's record, and the lse block inside it, 256-byte aligned


def shard_ranges(tok_begin: Sequence[int], tok_end: Sequence[int], world_size: int,
                 chunk_tokens: int) -> Tuple[List[List[int]], List[List[int]]]:
    """Split every sequence's slice ``[tok_begin[b], tok_end[b])`` into ``world_size`` consecutive ranges.

    Cuts fall on the absolute chunk grid (multiples of ``chunk_tokens``), so a chunk is never shared by
    two ranks and every rank's first page is whole; chunks are dealt out as evenly as their count
    allows, older tokens to lower ranks.  Returns ``(begins, ends)``, each ``[world_size][B]``; a rank
    with no chunk of a sequence gets an empty range there.
    """
    if world_size < 1 or chunk_tokens < 1:
        raise ValueError("world_size and chunk_tokens must be positive")
    begins = [[0] * len(tok_begin) for _ in range(world_size)]
    ends = [[0] * len(tok_begin) for _ in range(world_size)]
    for b, (tb, te) in enumerate(zip(tok_begin, tok_end)):
        tb, te = int(tb), int(te)
        if te < tb:
            raise ValueError("tok_end < tok_begin")
        first = tb // chunk_tokens
        n_chunks = 0 if te == tb else -(-te // chunk_tokens) - first
        for r in range(world_size):
            c0 = first + (n_chunks * r) // world_size
            c1 = first + (n_chunks * (r + 1)) // world_size
            lo = min(max(c0 * chunk_tokens, tb), te)
            hi = min(max(c1 * chunk_tokens, tb), te)
            begins[r][b], ends[r][b] = lo, hi
    return begins, ends


def record_floats(batch: int, num_q_heads: int, head_dim: int) -> int:
    """Length, in floats, of one rank's exchanged record: out [B][Hq][D], then lse [B][Hq], padded."""
    n = batch * num_q_heads * (head_dim + 1)
    return -(-n // RECORD_ALIGN) * RECORD_ALIGN


def pack_record(out: torch.Tensor, lse: torch.Tensor, record: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Copy a rank's merged ``out`` [B][Hq][D] and ``lse`` [B][Hq] into one flat fp32 record."""
    B, Hq, D = out.shape
    n = record_floats(B, Hq, D)
    if record is None:
        record = torch.zeros(n, dtype=torch.float32, device=out.device)
    elif record.numel() != n or record.dtype != torch.float32:
        raise ValueError("record has the wrong size or dtype")
    record[:B * Hq * D].copy_(out.reshape(-1))
    record[B * Hq * D:B * Hq * (D + 1)].copy_(lse.reshape(-1))
    return record


def exchange_records(record: torch.Tensor, group=None, gathered: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All-gather every rank's record into ``[world_size][record_floats]`` (rank order)."""
    world = dist.get_world_size(group)
    if gathered is None:
        gathered = torch.empty(world, record.numel(), dtype=record.dtype, device=record.device)
    dist.all_gather_into_tensor(gathered.view(-1), record, group=group)
    return gathered


def record_sources(gathered: torch.Tensor, batch: int, num_q_heads: int, head_dim: int,
                   ones: Optional[torch.Tensor] = None):
    """View the gathered records as ``world_size`` partial sources ``(o, m, l) = (out_r, lse_r, 1)``."""
    B, Hq, D = batch, num_q_heads, head_dim
    if ones is None:
        ones = torch.ones(B, Hq, 1, dtype=torch.float32, device=gathered.device)
    srcs = []
    for r in range(gathered.shape[0]):
        rec = gathered[r]
        srcs.append((rec[:B * Hq * D].view(B, Hq, 1, D), rec[B * Hq * D:B * Hq * (D + 1)].view(B, Hq, 1), ones))
    return srcs


class TokenShardedDecode:
    """One rank's side of a token-sharded decode step.

    ``tok_begin`` / ``tok_end`` are this rank's ranges (a row of ``shard_ranges``); the KV pool and block
    table hold this rank's pages.  ``step`` runs the local ``hg_attn_decode`` (with whatever host
    partials this rank was given), all-gathers the merged rows and merges them; every rank ends with the
    full result.  At most 8 ranks (the merge's source limit).
    """

    def __init__(self, desc: hg.HgAttnDesc, group=None, device=None):
        self.desc, self.group = desc, group
        self.world = dist.get_world_size(group) if dist.is_initialized() else 1
        if self.world > 8:
            raise ValueError("token sharding supports at most 8 ranks")
        B, Hq, D = desc.batch, desc.num_q_heads, desc.head_dim
        dev = torch.device(device if device is not None else "cuda")
        self.record = torch.zeros(record_floats(B, Hq, D), dtype=torch.float32, device=dev)
        self.local_out = self.record[:B * Hq * D].view(B, Hq, D)        # the local decode writes its rows
        self.local_lse = self.record[B * Hq * D:B * Hq * (D + 1)].view(B, Hq)   # straight into the record
        self.gathered = torch.empty(self.world, self.record.numel(), dtype=torch.float32, device=dev)
        self.ones = torch.ones(B, Hq, 1, dtype=torch.float32, device=dev)
        self.workspace = None

    def step(self, q, k_cache, v_cache, seq_lens, tok_begin, tok_end, host_partials, out, lse):
        d = self.desc
        need = hg.hg_attn_workspace_bytes(d, len(host_partials))
        if self.workspace is None or self.workspace.numel() < need:
            self.workspace = torch.empty(need, dtype=torch.uint8, device=self.record.device)
        hg.hg_attn_decode(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, host_partials, self.local_out,
                          self.local_lse, self.workspace, d)
        if self.world > 1 or dist.is_initialized():
            exchange_records(self.record, self.group, self.gathered)
        else:
            self.gathered[0].copy_(self.record)
        hg.hg_attn_merge(record_sources(self.gathered, d.batch, d.num_q_heads, d.head_dim, self.ones), out, lse, d)

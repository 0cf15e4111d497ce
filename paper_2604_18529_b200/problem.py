"""A workload materialised on one GPU: input tensors, output buffers and the ABI descriptor.

Shared by the tests, the smoke check and the bench so that all three call the library the same way.
Holds no attention arithmetic.
"""
from __future__ import annotations

from typing import List, Optional, Tuple

import torch

from . import binding as hg
from .workload import AttnWorkload


class DeviceProblem:
    def __init__(self, w: AttnWorkload, device="cuda:0", poison_tail: bool = False, kv: Optional[dict] = None,
                 flags: int = 0):
        self.w = w
        self.device = torch.device(device)
        dev = self.device
        self.kv = kv if kv is not None else w.build_device_kv(dev, poison_tail=poison_tail)
        self.q = w.q(dev)
        self.seq_lens = torch.tensor(w.seq_lens, dtype=torch.int32, device=dev)
        self.tok_begin = torch.tensor(w.tok_begin, dtype=torch.int32, device=dev)
        self.tok_end = torch.tensor(w.tok_end, dtype=torch.int32, device=dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.sched = torch.zeros(2, dtype=torch.int32, device=dev)
        self.NC = w.num_chunks
        self.desc = self.make_desc(w.chunk_tokens, self.NC, flags=flags)
        B, Hq, D, NC = w.B, w.Hq, w.D, self.NC
        self.o_part = torch.empty(B, Hq, NC, D, dtype=torch.float32, device=dev)
        self.m_part = torch.empty(B, Hq, NC, dtype=torch.float32, device=dev)
        self.l_part = torch.empty(B, Hq, NC, dtype=torch.float32, device=dev)
        self.out = torch.empty(B, Hq, D, dtype=torch.float32, device=dev)
        self.lse = torch.empty(B, Hq, dtype=torch.float32, device=dev)

    def make_desc(self, chunk_tokens: int, num_chunks: int, scale: float = 0.0, flags: int = 0, tune: int = 0,
                  tune_stages: int = 0, tune_ctas_per_sm: int = 0):
        w, kv = self.w, self.kv
        return hg.attn_desc(batch=w.B, num_q_heads=w.Hq, num_kv_heads=w.Hkv, head_dim=w.D, dtype=w.dtype,
                            page_size=w.page_size, num_pages=kv["num_pages"], page_stride=kv["page_stride"],
                            head_stride=kv["head_stride"], tok_stride=kv["tok_stride"], block_table=kv["block_table"],
                            max_pages=kv["max_pages"], chunk_tokens=chunk_tokens, num_chunks=num_chunks, scale=scale,
                            status=self.status, sched_counter=self.sched, flags=flags, tune=tune,
                            tune_stages=tune_stages, tune_ctas_per_sm=tune_ctas_per_sm)

    def partial(self, stream=None):
        hg.hg_attn_partial(self.q, self.kv["k"], self.kv["v"], self.seq_lens, self.tok_begin, self.tok_end,
                           self.o_part, self.m_part, self.l_part, self.desc, stream)

    def merge(self, host_partials: List[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]], stream=None):
        hg.hg_attn_merge([(self.o_part, self.m_part, self.l_part)] + list(host_partials), self.out, self.lse,
                         self.desc, stream)

    def step(self, host_partials, stream=None):
        """One pass of the whole path with inputs resident on the device."""
        self.partial(stream)
        self.merge(host_partials, stream)

    def prepare_step(self, host_partials, stream=None):
        """``step`` with the arguments of both calls marshalled once: a callable for timing loops and decode loops
        that keep their buffers.  Reflects the buffers and description as they are now."""
        partial = hg.prepare_partial(self.q, self.kv["k"], self.kv["v"], self.seq_lens, self.tok_begin, self.tok_end,
                                     self.o_part, self.m_part, self.l_part, self.desc, stream)
        merge = hg.prepare_merge([(self.o_part, self.m_part, self.l_part)] + list(host_partials), self.out, self.lse,
                                 self.desc, stream)

        def step() -> None:
            partial()
            merge()

        return step

    def alg_bytes(self) -> int:
        """Algorithmic bytes of one step: the slice's K and V once per KV head, plus q, the block-table
        entries of resident pages, the partials written and read back, and out/lse."""
        w = self.w
        rows = w.B * w.Hq
        nchunks = sum(w.chunk_grid(b)[1] for b in range(w.B))
        part = w.Hq * nchunks * (w.D + 2) * 4
        pages = self.kv["num_pages"] if w.paged else 0
        return w.kv_bytes() + rows * w.D * 2 + pages * 4 + 2 * part + rows * (w.D + 1) * 4

    def empty_host_partial(self, nc: int = 1):
        w, dev = self.w, self.device
        o = torch.zeros(w.B, w.Hq, nc, w.D, dtype=torch.float32, device=dev)
        m = torch.full((w.B, w.Hq, nc), float("-inf"), dtype=torch.float32, device=dev)
        l = torch.zeros(w.B, w.Hq, nc, dtype=torch.float32, device=dev)
        return o, m, l

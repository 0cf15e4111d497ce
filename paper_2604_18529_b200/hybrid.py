"""One layer's hybrid attention step as the paper runs it (Section 4.2 workflow, Section 4.3 scheduler).

The GPU attends the tokens it holds (``hg_attn_partial``) while the CPU stage runs beside it: it picks K
of the host-held tokens per (sequence, KV head) - Post-QK^T: logits of all host tokens, the K best;
Pre-QK^T: a position-based set, logits only for it - and ships those logits and the matching V rows.
The GPU turns them into softmax partials (``hg_attn_partial_from_logits``) and merges both sides
(``hg_attn_merge``).  The three measured latencies of a step (GPU stage, CPU stage, transfer) drive the
feedback scheduler (Algorithm 1), which sets K and the strategy of the next step.

This module is plumbing: buffers, two streams, events, clocks and calls.  All arithmetic is in the CUDA
library and the host library.  The CPU's query is an input here (the paper derives it from the previous
layer's input; that speculation is outside this package).
"""
from __future__ import annotations

import time
from dataclasses import dataclass
from typing import List, Optional

import torch

from . import binding as hg
from . import host as H

POST_QK, PRE_QK = 0, 1


@dataclass
class StepRecord:
    k: int                 # tokens per (sequence, KV head) the CPU stage handled in this step
    strategy: int          # POST_QK or PRE_QK
    t_gpu: float           # ms: the GPU's own partial kernel
    t_cpu: float           # ms: selection + logits + V-row gather on the host
    t_tx: float            # ms: host -> device copies of logits, V rows and counts
    t_step: float          # ms: wall clock of the whole step, results on the device


class HybridAttentionStep:
    """Buffers and control for repeated hybrid steps over one KV configuration.

    ``desc`` describes the GPU slice (as for ``hg_attn_partial``); ``k_host`` / ``v_host`` are the host-held
    rows ``[B][T][Hkv][D]`` (any strides, D contiguous) of which the first ``n_host[b]`` are valid.
    For batches that mix long and short sequences build ``desc`` with ``flags=HG_FLAG_SPARSE_EMPTY``: the
    chunk partials here are private to the step, so their empty slots need no zero-filled ``o`` rows.
    """

    def __init__(self, desc: hg.HgAttnDesc, k_host: torch.Tensor, v_host: torch.Tensor, n_host: torch.Tensor,
                 k_min: int, k_max: int, k_step: int, sinks: int = 4, handoff_chunk: int = 256, host_threads: int = 0,
                 overlap_transfer: bool = True, device="cuda"):
        self.desc, self.k_host, self.v_host, self.n_host = desc, k_host, v_host, n_host.to(torch.int32).contiguous()
        self.dev = torch.device(device)
        self.B, self.Hq, self.Hkv, self.D = desc.batch, desc.num_q_heads, desc.num_kv_heads, desc.head_dim
        self.G = self.Hq // self.Hkv
        self.dtype = k_host.dtype
        self.sinks, self.chunk, self.threads = sinks, handoff_chunk, host_threads
        # True: the copies start as soon as the CPU stage has its data, beside the partial kernel if that is still
        # running; False: they wait for it.  Measured on the OPT-13B shape the two differ by under 2 %.
        self.overlap_transfer = overlap_transfer
        self.k_max = k_max
        self.sched = H.FeedbackScheduler(k_min, k_max, k_step)
        self.k, self.strategy = k_min, POST_QK
        self.capacity = k_host.shape[1]                 # host rows per sequence the buffers are sized for
        B, Hq, Hkv, D, NC = self.B, self.Hq, self.Hkv, self.D, desc.num_chunks
        dev = self.dev
        # GPU side
        self.o_part = torch.empty(B, Hq, NC, D, dtype=torch.float32, device=dev)
        self.m_part = torch.empty(B, Hq, NC, dtype=torch.float32, device=dev)
        self.l_part = torch.empty(B, Hq, NC, dtype=torch.float32, device=dev)
        ncs = -(-k_max // handoff_chunk)
        self.h_o = torch.empty(B * Hq * ncs * D, dtype=torch.float32, device=dev)
        self.h_m = torch.empty(B * Hq * ncs, dtype=torch.float32, device=dev)
        self.h_l = torch.empty(B * Hq * ncs, dtype=torch.float32, device=dev)
        self.d_logits = torch.empty(B * Hq * k_max, dtype=torch.float32, device=dev)
        self.d_vsel = torch.empty(B * Hkv * k_max * D, dtype=self.dtype, device=dev)
        self.d_nsel = torch.empty(B, dtype=torch.int32, device=dev)
        # host side (pinned: the copies are asynchronous)
        self.p_logits = torch.empty(B * Hq * k_max, dtype=torch.float32).pin_memory()
        self.p_vsel = torch.empty(B * Hkv * k_max * D, dtype=self.dtype).pin_memory()
        self.p_nsel = torch.empty(B, dtype=torch.int32).pin_memory()
        self.full_logits = torch.empty(B * Hq * max(self.capacity, 1), dtype=torch.float32)
        self.scores = torch.empty(B * Hkv * max(self.capacity, 1), dtype=torch.float32)
        self.idx: Optional[torch.Tensor] = None        # [B][Hkv][k] of the last step
        self.n_sel: Optional[torch.Tensor] = None      # [B]
        self.copy_stream = torch.cuda.Stream(device=dev)
        self.ev = {n: torch.cuda.Event(enable_timing=True) for n in ("g0", "g1", "t0", "t1", "h1")}
        self.history: List[StepRecord] = []
        self._plan_k, self._plan_pos, self._plan_n, self._ranking = -1, None, None, None
        self._pending = None
        self.set_host_tokens(self.n_host)

    def set_host_tokens(self, n_host: torch.Tensor) -> None:
        """The host now holds the first ``n_host[b]`` rows of every sequence (after an eviction, say)."""
        self.n_host = n_host.to(torch.int32).contiguous()
        self.n_host_max = int(self.n_host.max()) if self.n_host.numel() else 0
        if self.n_host_max > self.capacity:
            raise ValueError("more host tokens than the host rows hold")
        self.n_rows = self.n_host.repeat_interleave(self.Hkv).contiguous()
        self._plan_k = -1

    def set_pre_qk_ranking(self, ranking: Optional[torch.Tensor]) -> None:
        """A ranked candidate list for Pre-QK^T selection, most important first: int32 ``[B][Hkv][R]`` of host token
        indices, -1 padded at the end (Section 4.5: any predictor - positions, accumulated scores, head
        importance - reduces to such a list; the selector takes its first K entries).  ``None`` goes back to
        the built-in position rule (sinks + most recent host tokens)."""
        if ranking is not None:
            if ranking.dtype != torch.int32 or ranking.dim() != 3 or ranking.shape[:2] != (self.B, self.Hkv):
                raise ValueError("ranking must be int32 [B][Hkv][R]")
            ranking = ranking.contiguous()
        self._ranking = ranking
        self._plan_k = -1

    def set_operating_point(self, k: int, strategy: int) -> None:
        """Override what the scheduler decided (tests, warm starts); the scheduler carries on from here."""
        self.k, self.strategy = k, strategy
        self.sched.state.k, self.sched.state.strategy = k, strategy

    # ---- CPU stage ------------------------------------------------------------------------------------------
    def _cpu_stage(self, q_host: torch.Tensor, k: int):
        B, Hq, Hkv, D = self.B, self.Hq, self.Hkv, self.D
        logits = self.p_logits[:B * Hq * k].view(B, Hq, k)
        vsel = self.p_vsel[:B * Hkv * k * D].view(B, Hkv, k, D)
        n_sel = self.p_nsel
        if self._plan_k != k:                       # counts and the Pre-QK^T set depend on k alone: kept between steps
            n_post = torch.minimum(self.n_host, torch.tensor(k, dtype=torch.int32))
            n_pre = n_post.clone()
            pos = torch.full((B, Hkv, k), -1, dtype=torch.int32)
            if self._ranking is not None:
                pos, n_pre = H.hg_host_select_ranked(self._ranking, self.n_host, k)      # the first K of the caller's lists
            else:
                for b in range(B):
                    sel = H.hg_host_select_positions(int(self.n_host[b]), self.sinks, max(k - self.sinks, 0), k)
                    pos[b, :, : len(sel)] = sel
            self._plan_k, self._plan_pos, self._plan_n = k, pos, (n_post, n_pre)
        n_sel.copy_(self._plan_n[0 if self.strategy == POST_QK and self.n_host_max > 0 else 1])
        sel_desc = H.host_desc(self.k_host, Hq, k, scale=self.desc.scale, threads=self.threads)
        if self.strategy == POST_QK and self.n_host_max > 0:
            n_max = self.n_host_max
            full = self.full_logits[:B * Hq * n_max].view(B, Hq, n_max)
            scores = self.scores[:B * Hkv * n_max].view(B * Hkv, n_max)
            full_desc = H.host_desc(self.k_host, Hq, n_max, scale=self.desc.scale, threads=self.threads)
            H.hg_host_logits(q_host, self.k_host, None, self.n_host, full, full_desc)
            H.hg_host_group_scores(full.view(B * Hq, n_max), self.G, self.n_rows, scores)
            idx, _ = H.hg_host_select_topk(scores, self.n_rows, k)
            idx = idx.view(B, Hkv, k)
            H.hg_host_gather_logits(full, idx, n_sel, logits, sel_desc)
        else:
            idx = self._plan_pos
            H.hg_host_logits(q_host, self.k_host, idx, n_sel, logits, sel_desc)
        H.hg_host_gather_rows(self.v_host, idx, n_sel, vsel, sel_desc)
        self.idx, self.n_sel = idx, n_sel.clone()
        return logits, vsel, n_sel

    # ---- one step, in the three pieces a pipeline needs -------------------------------------------------------------
    def cpu_stage(self, q_host: torch.Tensor):
        """Selection, logits and V-row gather for the current (K, strategy); host only, may run on another thread
        while the GPU works on something else.  Returns what ``finish`` needs."""
        t0 = time.perf_counter()
        k = self.k
        logits, vsel, n_sel = self._cpu_stage(q_host, k)
        return k, logits, vsel, n_sel, (time.perf_counter() - t0) * 1e3

    def launch_gpu(self, q_dev, k_cache, v_cache, seq_lens, tok_begin, tok_end) -> None:
        """The GPU stage: partials of the GPU-resident tokens, enqueued on the current stream."""
        main = torch.cuda.current_stream(self.dev)
        self.ev["g0"].record(main)
        hg.hg_attn_partial(q_dev, k_cache, v_cache, seq_lens, tok_begin, tok_end, self.o_part, self.m_part, self.l_part,
                           self.desc, main)
        self.ev["g1"].record(main)

    def finish(self, staged, out, lse) -> None:
        """Transfer of the CPU stage's output, hand-off partials (second stream) and the merge (current stream);
        everything is enqueued, nothing waited for."""
        B, Hq, Hkv, D = self.B, self.Hq, self.Hkv, self.D
        k, logits, vsel, n_sel, t_cpu = staged
        ev = self.ev
        main = torch.cuda.current_stream(self.dev)
        ld = hg.logits_desc(batch=B, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, dtype=self.dtype, max_selected=k,
                            chunk_tokens=self.chunk)
        ncs = ld.num_chunks
        d_logits = self.d_logits[:B * Hq * k].view(B, Hq, k)
        d_vsel = self.d_vsel[:B * Hkv * k * D].view(B, Hkv, k, D)
        h_o = self.h_o[:B * Hq * ncs * D].view(B, Hq, ncs, D)
        h_m = self.h_m[:B * Hq * ncs].view(B, Hq, ncs)
        h_l = self.h_l[:B * Hq * ncs].view(B, Hq, ncs)
        cs = self.copy_stream
        with torch.cuda.stream(cs):
            if not self.overlap_transfer:
                cs.wait_event(ev["g1"])
            ev["t0"].record(cs)
            d_logits.copy_(logits, non_blocking=True)
            d_vsel.copy_(vsel, non_blocking=True)
            self.d_nsel.copy_(n_sel, non_blocking=True)
            ev["t1"].record(cs)
            hg.hg_attn_partial_from_logits(d_logits, d_vsel, self.d_nsel, h_o, h_m, h_l, ld, cs)
            ev["h1"].record(cs)
        main.wait_event(ev["h1"])
        hg.hg_attn_merge([(self.o_part, self.m_part, self.l_part), (h_o, h_m, h_l)], out, lse, self.desc, main)
        self._pending = (k, self.strategy, t_cpu)

    def collect(self, t_step_ms: float = 0.0, update: bool = True) -> StepRecord:
        """After the stream has been synchronised: the step's record; with ``update`` Algorithm 1 moves (K, strategy)."""
        k, strategy, t_cpu = self._pending
        ev = self.ev
        rec = StepRecord(k=k, strategy=strategy, t_gpu=ev["g0"].elapsed_time(ev["g1"]), t_cpu=t_cpu,
                         t_tx=ev["t0"].elapsed_time(ev["t1"]), t_step=t_step_ms)
        self.history.append(rec)
        if update:
            self.k, self.strategy = self.sched.update(rec.t_gpu, rec.t_cpu, rec.t_tx)
        return rec

    def step(self, q_dev, q_host, k_cache, v_cache, seq_lens, tok_begin, tok_end, out, lse) -> StepRecord:
        """One layer by itself: GPU stage enqueued first, the CPU stage runs beside it on this thread."""
        t_wall = time.perf_counter()
        self.launch_gpu(q_dev, k_cache, v_cache, seq_lens, tok_begin, tok_end)
        staged = self.cpu_stage(q_host)
        self.finish(staged, out, lse)
        torch.cuda.current_stream(self.dev).synchronize()
        return self.collect((time.perf_counter() - t_wall) * 1e3)       # Algorithm 1, for the next step


class HybridPipeline:
    """Several layers run the way the paper's timeline shows (Section 4.3, workflow step 1): while the GPU works
    on layer i, a host thread already runs the CPU stage of layer i + 1.  One ``HybridAttentionStep`` per layer
    (each with its own buffers); the per-layer queries are inputs - deriving layer i + 1's query from layer i's
    input is the paper's speculation, outside this package.  A single (K, strategy) serves all layers of a pass
    and is updated once per pass from the mean latencies.
    """

    def __init__(self, layers: List[HybridAttentionStep]):
        from concurrent.futures import ThreadPoolExecutor
        self.layers = layers
        self.pool = ThreadPoolExecutor(max_workers=1)

    def run(self, q_dev: List[torch.Tensor], q_host: List[torch.Tensor], kv: List[tuple], outs: List[tuple],
            pipelined: bool = True) -> float:
        """``kv[i] = (k_cache, v_cache, seq_lens, tok_begin, tok_end)``, ``outs[i] = (out, lse)``.  Returns the wall
        time of the pass in ms.  ``pipelined=False`` runs the same work layer after layer (for comparison)."""
        L = self.layers
        dev = L[0].dev
        k, strategy = L[0].k, L[0].strategy
        for e in L:
            e.set_operating_point(k, strategy)
        t0 = time.perf_counter()
        fut = self.pool.submit(L[0].cpu_stage, q_host[0]) if pipelined else None
        for i, e in enumerate(L):
            e.launch_gpu(q_dev[i], *kv[i])
            staged = fut.result() if pipelined else e.cpu_stage(q_host[i])
            if pipelined and i + 1 < len(L):
                fut = self.pool.submit(L[i + 1].cpu_stage, q_host[i + 1])     # overlaps layer i's GPU work and transfer
            e.finish(staged, *outs[i])
            if not pipelined:
                torch.cuda.current_stream(dev).synchronize()
        torch.cuda.current_stream(dev).synchronize()
        ms = (time.perf_counter() - t0) * 1e3
        recs = [e.collect(update=False) for e in L]
        mean = lambda f: sum(getattr(r, f) for r in recs) / len(recs)
        k, strategy = L[0].sched.update(mean("t_gpu"), mean("t_cpu"), mean("t_tx"))
        for e in L:
            e.set_operating_point(k, strategy)
        return ms


class HostKvStore:
    """The host tier of the cache: pinned rows ``k``, ``v`` ``[B][capacity][Hkv][D]`` holding, for every sequence,
    its oldest tokens in original order - row i is absolute token i, ``n[b]`` rows valid - i.e. the prefix
    ``[0, tok_begin[b])`` that the Eviction Engine (Section 4.2) has moved off the GPU."""

    def __init__(self, batch: int, capacity: int, num_kv_heads: int, head_dim: int, dtype: torch.dtype,
                 k_node: Optional[int] = None, v_node: Optional[int] = None):
        """``k_node`` / ``v_node``: NUMA nodes to bind the K rows and the V rows to (Section 4.4: keys, which the CPU
        reads, in CPU DRAM; values, which only travel to the GPU, in the far tier); ``None`` leaves the placement
        to the allocator.  Either way the rows are pinned."""
        shape = (batch, capacity, num_kv_heads, head_dim)
        self._tiers = []
        def rows(node):
            if node is None:
                return torch.zeros(shape, dtype=dtype).pin_memory()
            buf = H.TierBuffer(shape, dtype, node, register=True)
            self._tiers.append(buf)
            buf.tensor.zero_()
            return buf.tensor
        self.k = rows(k_node)
        self.v = rows(v_node)
        self.n = torch.zeros(batch, dtype=torch.int32)
        self.capacity = capacity

    def evict_from_gpu(self, k_cache, v_cache, tok_begin, tok_end, n_evict: List[int], desc: hg.HgAttnDesc,
                       freed: Optional[torch.Tensor] = None, n_freed: Optional[torch.Tensor] = None) -> None:
        """Move the oldest ``n_evict[b]`` tokens of every GPU slice here: ``hg_kv_evict`` into a device staging
        buffer, one device -> host copy per sequence to the end of that sequence's rows, counts advanced.
        ``n_evict`` must not exceed the slices (the caller knows its own ranges); returns when the rows are here."""
        B, dev = len(n_evict), k_cache.device
        max_evict = max(max(n_evict), 1)
        if any(int(self.n[b]) + n_evict[b] > self.capacity for b in range(B)):
            raise ValueError("host rows full")
        Hkv, D = self.k.shape[2], self.k.shape[3]
        k_out = torch.empty(B, max_evict, Hkv, D, dtype=self.k.dtype, device=dev)
        v_out = torch.empty_like(k_out)
        hg.hg_kv_evict(k_cache, v_cache, tok_begin, tok_end, torch.tensor(n_evict, dtype=torch.int32, device=dev), k_out, v_out,
                       freed, n_freed, desc)
        for b in range(B):
            n0, ne = int(self.n[b]), n_evict[b]
            if ne:
                self.k[b, n0:n0 + ne].copy_(k_out[b, :ne], non_blocking=True)
                self.v[b, n0:n0 + ne].copy_(v_out[b, :ne], non_blocking=True)
            self.n[b] = n0 + ne
        torch.cuda.current_stream(dev).synchronize()

    def begin_evict(self, k_cache, v_cache, tok_begin, tok_end, n_evict: List[int], desc: hg.HgAttnDesc,
                    freed: Optional[torch.Tensor] = None, n_freed: Optional[torch.Tensor] = None) -> "PendingEviction":
        """The same move, draining beside the attention of this decode step instead of in front of it.

        On the current stream only ``hg_kv_evict_begin`` is enqueued: it advances ``tok_begin``, so the attention the
        caller enqueues next already covers the shrunk slice.  The row copy, the device -> host copies and the
        un-mapping of the emptied pages (``hg_kv_evict_copy``, ``hg_kv_evict_finish``) go to this store's own stream
        behind an event.  Call ``wait()`` on the returned object before using the host rows or the freed pages."""
        B, dev = len(n_evict), k_cache.device
        max_evict = max(max(n_evict), 1)
        if any(int(self.n[b]) + n_evict[b] > self.capacity for b in range(B)):
            raise ValueError("host rows full")
        Hkv, D = self.k.shape[2], self.k.shape[3]
        if getattr(self, "_stream", None) is None:
            self._stream = torch.cuda.Stream(device=dev)
        main, side = torch.cuda.current_stream(dev), self._stream
        k_out = torch.empty(B, max_evict, Hkv, D, dtype=self.k.dtype, device=dev)
        v_out = torch.empty_like(k_out)
        src_begin = torch.empty(B, dtype=torch.int32, device=dev)
        n_moved = torch.empty(B, dtype=torch.int32, device=dev)
        n_dev = torch.tensor(n_evict, dtype=torch.int32, device=dev)
        hg.hg_kv_evict_begin(tok_begin, tok_end, n_dev, max_evict, 0 if freed is None else freed.shape[1], src_begin, n_moved,
                             desc, main)
        started = torch.cuda.Event()
        started.record(main)
        moved_host = torch.empty(B, dtype=torch.int32).pin_memory()
        with torch.cuda.stream(side):
            side.wait_event(started)
            hg.hg_kv_evict_copy(k_cache, v_cache, src_begin, n_moved, k_out, v_out, desc, side)
            for b in range(B):
                n0, ne = int(self.n[b]), n_evict[b]
                if ne:
                    self.k[b, n0:n0 + ne].copy_(k_out[b, :ne], non_blocking=True)
                    self.v[b, n0:n0 + ne].copy_(v_out[b, :ne], non_blocking=True)
            hg.hg_kv_evict_finish(src_begin, n_moved, freed, n_freed, desc, side)
            moved_host.copy_(n_moved, non_blocking=True)
            done = torch.cuda.Event()
            done.record(side)
        for t in (k_out, v_out, src_begin, n_moved, n_dev):
            t.record_stream(side)
        return PendingEviction(self, done, moved_host, list(n_evict))


class PendingEviction:
    """An eviction whose copies are still draining on the store's stream."""

    def __init__(self, store: HostKvStore, done: torch.cuda.Event, moved_host: torch.Tensor, asked: List[int]):
        self.store, self.done, self.moved_host, self.asked = store, done, moved_host, asked

    def wait(self) -> List[int]:
        """Blocks until the rows are in the host tier; returns how many rows of every sequence arrived (fewer than
        asked for only when the library cut a range back) and counts them in."""
        self.done.synchronize()
        moved = self.moved_host.tolist()
        for b, m in enumerate(moved):
            self.store.n[b] = int(self.store.n[b]) + m
        return moved


#!/usr/bin/env python
"""Benchmark of the hybrid decode-attention hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: hg_attn_partial over the
GPU-resident KV slice, then hg_attn_merge of the chunk partials with the partials of the host-held
slice.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME|all] [--repeats R] [--impl reference]

Without --workload the headline (value, roofline, e2e, cpu_baseline) is the largest single-GPU
configuration, `opt30b`, and `config.workloads` carries one record per configuration (the four
32K-1M-token ones with their roofline and end-to-end figures, `tiny` in microseconds only).  Every
workload's timed pass of K steps is repeated R times; the headline is the median repeat.

N > 1: one rank per GPU, each running its own copy of the workload (independent sequences, no
data-path collective): weak scaling.  Started without a launcher (no WORLD_SIZE in the environment)
the script starts its own N ranks through torch.distributed.run.  With N > 1 the line also carries
`sharded`: the 1M-token configuration cut by token range over the N ranks, the one mode of the path
with a real exchange step (an all-gather of one merged row per head into local memory).
"""
import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode attention KV tokens/s"
UNIT = "KV tokens/s"
FALLBACK_HBM_GBS = 6650.0
HEADLINE = "opt30b"                      # the largest configuration that fits one GPU (7.5 GB of KV per step)
LARGE = ("opt13b", "opt30b", "llama70b", "ragged")
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the partial kernel, one ncu capture per workload
# (absent until a capture of that workload exists).  Traffic grows in proportion to the tokens processed, so a
# capture of the first sequences is scaled to the full launch.
NCU_TRAFFIC_BYTES = {
    "opt13b": 4 * (805_556_224 + 4_392_704),          # two of the eight sequences captured, x 4
    "llama70b": 1_718_243_000 + 4_194_048,            # the full launch captured
    "opt30b": 4 * (1_879_137_000 + 3_563_520),        # one of the four sequences captured, x 4
    "ragged": 951_552_512 + 4_044_288,                # the full launch captured
}


def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of `values` over all ranks (identity when not running distributed)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(tokens_per_rank, world, ms_per_step):
    """KV tokens/s of the whole job: every rank processes its own copy of the workload (weak scaling),
    and the job is as slow as its slowest rank."""
    return world * tokens_per_rank / (ms_per_step * 1e-3)


def measured_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def launcher_command(args_list, n, port=None):
    """The command that starts `n` ranks of this script on this node (one per GPU)."""
    port = port or (29500 + os.getpid() % 1500)
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(args_list)


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed regions run."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def window(self, t0, t1, fallback_all=True):
        """Median SM clock, maximum clock and the throttle reasons seen between wall times t0 and t1."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        rows = [l for t, l in list(self.lines) if t0 - 0.03 <= t <= t1 + 0.05]
        if not rows and fallback_all:
            rows = [l for _, l in list(self.lines)]
        sm, mx, reasons = [], [], set()
        for l in rows:
            p = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except Exception:
                continue
            for n, v in zip(self.NAMES, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass


def oracle_sample(w, rows_budget, device):
    """Inputs for the oracle's share of the work: the GPU slice of `rows_budget` (sequence, head) rows."""
    import numpy as np
    import torch
    rows = []
    for b in range(w.B):
        for h in range(w.Hq):
            if len(rows) < rows_budget and w.tok_end[b] > w.tok_begin[b]:
                rows.append((b, h))
    bits = lambda t: t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    qall = w.q()
    items = []
    for b, h in rows:
        g = h // w.G
        K = bits(w.kv_rows("k", b, g, w.tok_begin[b], w.tok_end[b], device))
        V = bits(w.kv_rows("v", b, g, w.tok_begin[b], w.tok_end[b], device))
        items.append((bits(qall[b, h]), K, V, w.tok_begin[b], w.tok_end[b]))
    tokens = sum(it[4] - it[3] for it in items) / w.Hq     # in units of whole-layer token positions
    return items, tokens


def oracle_pass(w, items, threads):
    """PARTIAL per chunk over each sampled row's slice, then MERGE (the same work the GPU path does)."""
    from concurrent.futures import ThreadPoolExecutor
    from oracle import hg_oracle as O
    C = w.chunk_tokens

    def one(it):
        q, K, V, tb, te = it
        n = te - tb
        NC = -(-te // C) - tb // C
        # a row is its own one-sequence, one-head cache whose token 0 is the slice's first token;
        # the chunk grid is shifted accordingly so that chunks sit on the same absolute boundaries
        off = tb % C
        m, l, o = O.chunked_partials(q.reshape(1, 1, -1), _pad(K, off).reshape(1, n + off, 1, -1),
                                     _pad(V, off).reshape(1, n + off, 1, -1), w.dtype, [off], [n + off], C, NC, threads=1)
        return O.merge(m[0, 0], l[0, 0], o[0, 0])

    with ThreadPoolExecutor(max_workers=threads) as ex:      # the C calls release the GIL
        return list(ex.map(one, items))


def _pad(a, off):
    import numpy as np
    if off == 0:
        return a
    return np.concatenate([np.zeros((off, a.shape[1]), dtype=a.dtype), a], axis=0)


def time_oracle(w, device, target_core_seconds=20.0):
    from oracle import hg_oracle as O
    threads = O.host_threads()
    per_row = 0.17 * (sum(e - b for b, e in zip(w.tok_begin, w.tok_end)) / max(1, w.B)) / 19660.0 * (w.D / 128.0)
    budget = max(threads, min(w.B * w.Hq, int(target_core_seconds / max(per_row, 1e-6))))
    items, tokens = oracle_sample(w, budget, device)
    t0 = time.perf_counter()
    oracle_pass(w, items, threads)
    dt = time.perf_counter() - t0
    return {"value": tokens / dt, "unit": UNIT, "cores": threads, "kind": "oracle", "workload": w.name,
            "sample": f"{len(items)} of {w.B * w.Hq} (sequence, head) rows, full GPU slice each, "
                      f"chunked PARTIAL + MERGE in fp64, {dt:.2f} s"}, items, tokens


def time_extras(w, prob, dev, steps):
    """The widened entry points on the same shapes: the CPU -> GPU hand-off (K_sel selected host tokens per
    sequence), the host logits calculator feeding it, and the residency operations."""
    import statistics as st
    import torch
    import paper_2604_18529_b200 as pkg
    from paper_2604_18529_b200 import host as H

    def dev_us(fn, n):
        for _ in range(3):
            fn()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for a, b in ev:
            a.record(); fn(); b.record()
        torch.cuda.synchronize()
        return st.mean(a.elapsed_time(b) for a, b in ev) * 1e3

    out = {}
    dt = {"f16": torch.float16, "bf16": torch.bfloat16}[w.dtype]
    gen = torch.Generator(device=dev).manual_seed(7)
    # ---- hand-off: logits [B][Hq][K] + V rows [B][Hkv][K][D] -> partials
    K_sel, chunk = 1024, 256
    logits = torch.randn(w.B, w.Hq, K_sel, device=dev, generator=gen)
    vrows = torch.randn(w.B, w.Hkv, K_sel, w.D, device=dev, generator=gen).to(dt)
    n_sel = torch.full((w.B,), K_sel, dtype=torch.int32, device=dev)
    ld = pkg.logits_desc(batch=w.B, num_q_heads=w.Hq, num_kv_heads=w.Hkv, head_dim=w.D, dtype=w.dtype, max_selected=K_sel,
                         chunk_tokens=chunk)
    ho = torch.empty(w.B, w.Hq, ld.num_chunks, w.D, device=dev); hm = torch.empty(w.B, w.Hq, ld.num_chunks, device=dev)
    hl = torch.empty_like(hm)
    us = dev_us(lambda: pkg.hg_attn_partial_from_logits(logits, vrows, n_sel, ho, hm, hl, ld), steps)
    nbytes = logits.numel() * 4 + vrows.numel() * 2
    out["handoff"] = {"selected_per_seq": K_sel, "us": us, "gbs": nbytes / us / 1e3}
    # ---- host logits calculator: every host-held token of the first sequence(s), all heads
    n_host = min(w.tok_begin[0], 16384)
    if n_host > 0:
        Bh = min(w.B, 2)
        k_host = torch.randn(Bh, n_host, w.Hkv, w.D).to(dt)
        q_host = torch.randn(Bh, w.Hq, w.D).to(dt)
        lg = torch.empty(Bh, w.Hq, n_host)
        nh = torch.full((Bh,), n_host, dtype=torch.int32)
        d = H.host_desc(k_host, w.Hq, n_host)
        H.hg_host_logits(q_host, k_host, None, nh, lg, d)
        t0 = time.perf_counter()
        reps = 3
        for _ in range(reps):
            H.hg_host_logits(q_host, k_host, None, nh, lg, d)
        sec = (time.perf_counter() - t0) / reps
        out["host_logits"] = {"tokens": Bh * n_host, "q_heads": w.Hq, "ms": sec * 1e3,
                              "gflops": 2.0 * Bh * n_host * w.Hq * w.D / sec / 1e9,
                              "k_gbs": Bh * n_host * w.Hkv * w.D * 2 / sec / 1e9, "cores": len(os.sched_getaffinity(0))}
    # ---- the whole hybrid step with Algorithm 1 in the loop: GPU slice + up to 8192 host-held tokens per sequence,
    #      of which the scheduler lets the CPU stage hand K over
    n_h = min(min(w.tok_begin), 8192)
    if n_h >= 512:
        from paper_2604_18529_b200 import hybrid
        kh = torch.randn(w.B, n_h, w.Hkv, w.D).to(dt); vh = torch.randn(w.B, n_h, w.Hkv, w.D).to(dt)
        qh = prob.q.cpu()
        eng = hybrid.HybridAttentionStep(prob.desc, kh, vh, torch.full((w.B,), n_h, dtype=torch.int32), k_min=128, k_max=1024,
                                         k_step=128, sinks=4, device=dev)
        with torch.cuda.device(dev):
            recs = [eng.step(prob.q, qh, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                             prob.out, prob.lse) for _ in range(12)]
        out["hybrid_step"] = {"host_tokens_per_seq": n_h, "k_min": 128, "k_max": 1024, "k_step": 128,
                              "steps": [{"k": r.k, "strategy": "post_qk" if r.strategy == 0 else "pre_qk",
                                         "t_gpu_ms": round(r.t_gpu, 3), "t_cpu_ms": round(r.t_cpu, 3),
                                         "t_tx_ms": round(r.t_tx, 3), "t_step_ms": round(r.t_step, 3)} for r in recs]}
        # the same step for 8 layers (one cache, a query per layer): layer after layer, and with the CPU stage of layer
        # i + 1 on a host thread while the GPU handles layer i (the paper's pipelined execution)
        L = 8
        layers = [hybrid.HybridAttentionStep(prob.desc, kh, vh, torch.full((w.B,), n_h, dtype=torch.int32), k_min=128,
                                             k_max=1024, k_step=128, sinks=4, device=dev) for _ in range(L)]
        pipe = hybrid.HybridPipeline(layers)
        qd = [prob.q] * L
        qhs = [qh] * L
        kvs = [(prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end)] * L
        outs = [(torch.empty_like(prob.out), torch.empty_like(prob.lse)) for _ in range(L)]
        times = {}
        with torch.cuda.device(dev):
            for mode in (False, True):
                best = None
                for _ in range(6):
                    for e in layers:
                        e.set_operating_point(128, hybrid.PRE_QK)
                    ms = pipe.run(qd, qhs, kvs, outs, pipelined=mode)
                    best = ms if best is None else min(best, ms)
                times[mode] = best
        out["hybrid_pipeline"] = {"layers": L, "k": 128, "strategy": "pre_qk", "layer_after_layer_ms": round(times[False], 3),
                                  "pipelined_ms": round(times[True], 3)}
        del eng, kh, vh, layers, pipe
    # ---- residency: evict 1024 oldest tokens per sequence into staging (state is restored between runs)
    max_evict = 1024
    k_out = torch.empty(w.B, max_evict, w.Hkv, w.D, dtype=dt, device=dev); v_out = torch.empty_like(k_out)
    ne = torch.full((w.B,), max_evict, dtype=torch.int32, device=dev)
    tb0 = prob.tok_begin.clone()
    table0 = None if prob.kv["block_table"] is None else prob.kv["block_table"].clone()

    def evict():
        prob.tok_begin.copy_(tb0)
        if table0 is not None:
            prob.kv["block_table"].copy_(table0)
        pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, ne, k_out, v_out, None, None, prob.desc)

    def restore_only():
        prob.tok_begin.copy_(tb0)
        if table0 is not None:
            prob.kv["block_table"].copy_(table0)

    us = dev_us(evict, steps) - dev_us(restore_only, steps)
    restore_only()
    moved = 2 * 2 * w.B * max_evict * w.Hkv * w.D * 2                 # K and V, read + written
    out["kv_evict"] = {"tokens_per_seq": max_evict, "us": us, "gbs": moved / us / 1e3}
    # ---- the same eviction with the step's attention: in front of it on one stream, and beside it (three-step form:
    #      begin on the attention's stream, row copy + device -> host copies + un-mapping on a second stream)
    kh = torch.empty(k_out.shape, dtype=dt).pin_memory(); vh = torch.empty_like(kh).pin_memory()
    src_begin = torch.empty(w.B, dtype=torch.int32, device=dev); n_moved = torch.empty_like(src_begin)
    side = torch.cuda.Stream(device=dev)
    main = torch.cuda.current_stream(dev)
    step = prob.prepare_step([prob.empty_host_partial()])

    def serial():
        restore_only()
        pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, ne, k_out, v_out, None, None, prob.desc)
        kh.copy_(k_out, non_blocking=True); vh.copy_(v_out, non_blocking=True)
        step()

    def beside():
        restore_only()
        pkg.hg_kv_evict_begin(prob.tok_begin, prob.tok_end, ne, max_evict, 0, src_begin, n_moved, prob.desc)
        ev = torch.cuda.Event(); ev.record(main)
        with torch.cuda.stream(side):
            side.wait_event(ev)
            pkg.hg_kv_evict_copy(prob.kv["k"], prob.kv["v"], src_begin, n_moved, k_out, v_out, prob.desc, side)
            kh.copy_(k_out, non_blocking=True); vh.copy_(v_out, non_blocking=True)
            pkg.hg_kv_evict_finish(src_begin, n_moved, None, None, prob.desc, side)
            fin = torch.cuda.Event(); fin.record(side)
        step()
        main.wait_event(fin)                  # the timed region ends when both the attention and the eviction are done

    base = dev_us(restore_only, steps)
    out["evict_with_attention"] = {"tokens_per_seq": max_evict, "d2h_bytes": 2 * kh.numel() * 2,
                                   "in_front_us": dev_us(serial, steps) - base, "beside_us": dev_us(beside, steps) - base,
                                   "attention_alone_us": dev_us(step, steps)}
    restore_only()
    return out


def time_handoff(dev, steps):
    """The device side of the paper's literal hand-off on HBM-resident inputs larger than L2: partials from host-computed
    logits [B][Hq][K] and V rows [B][Hkv][K][D] (hg_attn_partial_from_logits), one head per KV head and groups of 8."""
    import torch
    import paper_2604_18529_b200 as pkg
    peak, peak_kind = measured_peak()
    out = []
    # 256-slot chunks go to the warp-level kernel, 512-slot chunks to the tcgen05 kernel (the library's choice)
    for name, B, Hq, Hkv, K, chunk in (("mha", 8, 40, 40, 8192, 256), ("gqa8", 1, 64, 8, 262144, 256),
                                       ("mha_c512", 8, 40, 40, 8192, 512), ("gqa8_c512", 1, 64, 8, 262144, 512)):
        gen = torch.Generator(device=dev).manual_seed(11)
        logits = torch.randn(B, Hq, K, device=dev, generator=gen)
        vrows = torch.randn(B, Hkv, K, 128, device=dev, generator=gen).half()
        n_sel = torch.full((B,), K, dtype=torch.int32, device=dev)
        ld = pkg.logits_desc(batch=B, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=128, dtype="f16", max_selected=K, chunk_tokens=chunk)
        o = torch.empty(B, Hq, ld.num_chunks, 128, device=dev); m = torch.empty(B, Hq, ld.num_chunks, device=dev); l = torch.empty_like(m)
        call = lambda: pkg.hg_attn_partial_from_logits(logits, vrows, n_sel, o, m, l, ld)
        for _ in range(3):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        us = e0.elapsed_time(e1) * 1e3 / steps
        nbytes = logits.numel() * 4 + vrows.numel() * 2 + o.numel() * 4 + 2 * m.numel() * 4
        out.append({"shape": name, "batch": B, "q_heads": Hq, "kv_heads": Hkv, "head_dim": 128, "selected_per_seq": K,
                    "chunk_tokens": chunk, "kernel": "tcgen05.mma, accumulator in tensor memory" if chunk >= 512 else "mma.sync",
                    "us": us, "alg_bytes": nbytes, "gbs": nbytes / us / 1e3,
                    "frac": nbytes / us / 1e3 / peak, "peak_kind": f"{peak_kind} copy bandwidth",
                    "frac_of_8000": nbytes / us / 1e3 / 8000.0})
        del logits, vrows, o, m, l
    torch.cuda.empty_cache()
    return out


def run_reference(args, rank, world):
    """--impl reference: the fp64 oracle on the host cores, each step a bounded sample of the workload."""
    if rank != 0:
        return
    import torch
    from oracle import hg_oracle as O
    from paper_2604_18529_b200 import workload as W
    name = HEADLINE if args.workload in (None, "all") else args.workload
    w = W.make_workload(name)
    dev = "cuda:0" if torch.cuda.is_available() else "cpu"
    threads = O.host_threads()
    items, tokens = oracle_sample(w, max(threads, 16), dev)
    for _ in range(min(args.warmup, 1)):
        oracle_pass(w, items[:threads], threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_pass(w, items, threads)
    dt = (time.perf_counter() - t0) / args.steps
    value = tokens / dt
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": name, "sample": f"{len(items)} of {w.B * w.Hq} (sequence, head) rows per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{len(items)} rows x {args.steps} steps"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


class Ranks:
    """This process's place in the job, its device and the barrier every timed region is bracketed by."""

    def __init__(self, rank, local_rank, world):
        self.rank, self.local_rank, self.world = rank, local_rank, world
        self.dev = f"cuda:{local_rank}"

    def barrier(self):
        import torch
        import torch.distributed as dist
        torch.cuda.synchronize()
        if self.world > 1:
            dist.barrier()
        torch.cuda.synchronize()


def measure_workload(name, args, R, sampler):
    """All timings of one workload on this rank's GPU; times are the maximum over ranks.  Returns the record of
    `config.workloads` plus, under "_headline", what the top-level keys need (rank 0 only reads it)."""
    import torch
    import paper_2604_18529_b200 as pkg
    from paper_2604_18529_b200 import workload as W
    from paper_2604_18529_b200.problem import DeviceProblem

    dev, K = R.dev, args.steps
    w = W.make_workload(name)
    if args.batch:
        w = W.first_sequences(w, args.batch)
    if args.chunk:
        import dataclasses
        w = dataclasses.replace(w, chunk_tokens=args.chunk)
    # (empty chunk slots - a ragged batch has many - get m = -inf and l = 0 only: the merge never reads their o rows;
    # the work counter starts at zero and every call leaves it so: no clearing between the steps of the loop)
    prob = DeviceProblem(w, dev, flags=pkg.binding.HG_FLAG_SPARSE_EMPTY | pkg.binding.HG_FLAG_COUNTER_CLEAN)
    # partials of the host-held slice: produced by the host in the real system; here synthetic values with
    # the statistics of a real partial (they are inputs of the merge, not results of this library)
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    host = [(torch.randn(w.B, w.Hq, 1, w.D, device=dev, generator=gen),
             torch.randn(w.B, w.Hq, 1, device=dev, generator=gen),
             torch.rand(w.B, w.Hq, 1, device=dev, generator=gen) + 1.0)]
    stream = torch.cuda.current_stream()
    step = prob.prepare_step(host)          # both calls with their arguments marshalled once, as a decode loop would
    torch.cuda.synchronize()
    time.sleep(0.5)                         # input generation is heavy integer work: let the power average settle
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if int(prob.status.item()) != 0:
        raise SystemExit(f"{name}: device status {int(prob.status.item())} after warm-up")

    # ---- pass A: exactly K steps between one pair of events, repeated ----------------------------------------
    reps = []
    for _ in range(max(1, args.repeats)):
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        R.barrier()
        t0 = time.time()
        ev0.record(stream)
        for _ in range(K):
            step()
        ev1.record(stream)
        R.barrier()
        t1 = time.time()
        reps.append((ev0.elapsed_time(ev1), t0, t1))
    rep_ms = max_over_ranks([r[0] for r in reps], dev)
    order = sorted(range(len(rep_ms)), key=lambda i: rep_ms[i])
    med = order[(len(order) - 1) // 2]       # the median repeat (the lower one of an even count)
    ms_step = rep_ms[med] / K

    # the read probe: the partial kernel's own loads (same boxes, same ring, same schedule) with no arithmetic - what
    # this access pattern can reach; K launches back to back between one pair of events, like the steps of pass A,
    # and right after them (the board is then in the state the steps were timed in)
    probe_us = None
    if (w.kv_bytes() > 2 * 126e6 and not args.no_probe) or args.probe:
        sink = torch.zeros(w.B, w.Hkv, prob.NC, dtype=torch.int32, device=dev)
        probe = lambda: pkg.hg_kv_read_probe(prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, sink, prob.desc)
        for _ in range(3):
            probe()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        p0.record(stream)
        for _ in range(K):
            probe()
        p1.record(stream)
        torch.cuda.synchronize()
        probe_us = p0.elapsed_time(p1) * 1e3 / K

    # ---- pass B: K more steps with an event around every kernel (roofline of the dominant kernel) ----------
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    tb0 = time.time()
    for e in evs:
        e[0].record(stream); prob.partial(); e[1].record(stream); prob.merge(host); e[2].record(stream)
    torch.cuda.synchronize()
    tb1 = time.time()
    part_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    merge_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)

    # ---- one step at a time: nothing of a step overlaps its neighbours (in the loop above the merge and the next
    #      partial kernel start inside their predecessors' tails and the next step's first tiles are requested early)
    iso = []
    for _ in range(min(K, 20)):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream); step(); b.record(stream)
        torch.cuda.synchronize()
        iso.append(a.elapsed_time(b))
    (iso_ms,) = max_over_ranks([statistics.median(iso)], dev)

    # ---- end to end: per-step data in pinned host memory, results read back every step -----------------------
    pin = lambda t: t.cpu().pin_memory()
    q_h, sl_h, tb_h, te_h = pin(prob.q), pin(prob.seq_lens), pin(prob.tok_begin), pin(prob.tok_end)
    host_h = [tuple(pin(x) for x in src) for src in host]
    out_h = torch.empty(prob.out.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(prob.lse.shape, dtype=torch.float32).pin_memory()
    ws = torch.zeros(pkg.hg_attn_workspace_bytes(prob.desc, 1), dtype=torch.uint8, device=dev)   # (zero-filled: see HG_FLAG_COUNTER_CLEAN)
    decode_host = pkg.prepare_decode_host(q_h, prob.kv["k"], prob.kv["v"], sl_h, tb_h, te_h, host_h, out_h, lse_h, ws,
                                          prob.desc)     # arguments marshalled once, as a decode loop would

    def e2e_step():
        decode_host()
        stream.synchronize()            # the caller reads out_h / lse_h after every step

    for _ in range(3):
        e2e_step()
    R.barrier()
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record(stream)
    for _ in range(K):
        e2e_step()
    ee1.record(stream)
    R.barrier()
    (e2e_ms,) = max_over_ranks([ee0.elapsed_time(ee1)], dev)
    same = torch.equal(out_h, prob.out.cpu()) and torch.equal(lse_h, prob.lse.cpu())
    h2d = sum(t.numel() * t.element_size() for t in (q_h, sl_h, tb_h, te_h)) + \
        sum(t.numel() * t.element_size() for src in host_h for t in src)
    d2h = out_h.numel() * 4 + lse_h.numel() * 4

    extras = time_extras(w, prob, dev, K) if args.extras and R.rank == 0 and name != "tiny" else None
    if int(prob.status.item()) != 0:
        raise SystemExit(f"{name}: device status {int(prob.status.item())} after the timed passes")

    tokens = w.gpu_tokens
    kv_bytes = w.kv_bytes()
    large = kv_bytes > 2 * 126e6
    peak, peak_kind = measured_peak()
    nchunks = sum(w.chunk_grid(b)[1] for b in range(w.B))
    part_alg = kv_bytes + w.B * w.Hq * w.D * 2 + (prob.kv["num_pages"] * 4 if w.paged else 0) + w.Hq * nchunks * (w.D + 2) * 4
    achieved = part_alg / (part_ms * 1e-3) / 1e9
    step_gbs = prob.alg_bytes() / (ms_step * 1e-3) / 1e9
    clocks_med = sampler.window(reps[med][1], reps[med][2]) if sampler else None
    rec = {
        "workload": w.name, "batch": w.B, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": w.D, "kv_dtype": w.dtype,
        "context": max(w.seq_lens), "gpu_tokens": tokens, "page_size": w.page_size, "chunk_tokens": w.chunk_tokens,
        "kv_bytes_per_step": kv_bytes,
        "l2": "inputs larger than L2" if large else "inputs fit L2: launch-bound case, microseconds only",
        "us_per_step": ms_step * 1e3, "ms_per_step": ms_step,
        "repeats_ms_per_step": {"median": ms_step, "min": min(rep_ms) / K, "max": max(rep_ms) / K,
                                "all": [m / K for m in rep_ms],
                                "sm_mhz": [sampler.window(r[1], r[2], fallback_all=False)["sm_mhz"] if sampler else None
                                           for r in reps]},
        "kv_tokens_per_s": whole_job_value(tokens, R.world, ms_step),
        "partial_us": part_ms * 1e3, "merge_us": merge_ms * 1e3, "isolated_step_us": iso_ms * 1e3,
        "kernel_timing": "a second pass of K steps with CUDA events around each kernel; those events keep the merge "
                         "from starting as a programmatic dependent inside the partial kernel's tail, so partial_us + "
                         "merge_us can exceed the step time of the first pass",
        "probe_us": probe_us, "extras": extras,
        "clocks": clocks_med,
        "e2e": {"value": whole_job_value(tokens, R.world, e2e_ms / K), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / K, "matches_device_path": bool(same),
                "api": "hg_attn_decode_host via prepare_decode_host (KV pools stay device resident: they are the "
                       "GPU's slice of the cache)"},
    }
    if large:
        rec["step_gbs"] = step_gbs
        rec["step_frac_of_8000"] = step_gbs / 8000.0
        rec["step_frac_of_probe"] = probe_us / (ms_step * 1e3) if probe_us else None
        rec["probe"] = ("hg_kv_read_probe: the partial kernel's loads with every word XOR-folded instead of the attention "
                        "arithmetic, K launches back to back right after the timed steps")
        rec["roofline"] = {"bound": "hbm", "kernel": "partial_kernel", "achieved": achieved, "peak": peak,
                           "peak_kind": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                           "frac_of_8000": achieved / 8000.0, "alg_bytes_per_launch": part_alg,
                           "traffic": None if args.batch else NCU_TRAFFIC_BYTES.get(name)}
    else:
        # the contract asks for a roofline object on every line; for a launch-bound case it is context only
        rec["roofline"] = {"bound": "hbm", "kernel": "partial_kernel", "achieved": achieved, "peak": peak,
                           "peak_kind": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                           "frac_of_8000": achieved / 8000.0, "alg_bytes_per_launch": part_alg, "traffic": None,
                           "note": "launch-bound: the inputs fit L2"}
    rec["_headline"] = {"w": w, "ms_step": ms_step, "tokens": tokens, "wall": (reps[0][1], tb1)}
    del prob, ws, host
    torch.cuda.empty_cache()
    return rec


def measure_sharded(args, R):
    """The 1M-token configuration cut by token range over the ranks: local decode over this rank's range, one
    all-gather of a merged row per (sequence, head) into local memory, local merge.  Times are max over ranks."""
    import dataclasses
    import torch
    import torch.distributed as dist
    from paper_2604_18529_b200 import sharded, workload as W
    from paper_2604_18529_b200.problem import DeviceProblem

    dev, K = R.dev, args.steps
    w = W.make_workload("llama70b")
    begins, ends = sharded.shard_ranges(w.tok_begin, w.tok_end, R.world, w.chunk_tokens)
    mine = dataclasses.replace(w, name=f"llama70b[rank {R.rank}/{R.world}]", tok_begin=begins[R.rank], tok_end=ends[R.rank])
    prob = DeviceProblem(mine, dev)          # only this rank's pages are resident
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    host = [(torch.randn(w.B, w.Hq, 1, w.D, device=dev, generator=gen),
             torch.randn(w.B, w.Hq, 1, device=dev, generator=gen),
             torch.rand(w.B, w.Hq, 1, device=dev, generator=gen) + 1.0)] if R.rank == 0 else []
    eng = sharded.TokenShardedDecode(prob.desc, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        eng.step(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, host, prob.out, prob.lse)

    for _ in range(max(3, args.warmup)):
        step()
    R.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(K):
        step()
    e1.record(stream)
    R.barrier()
    x0, x1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    x0.record(stream)
    for _ in range(K):
        if dist.is_initialized():
            sharded.exchange_records(eng.record, None, eng.gathered)
    x1.record(stream)
    R.barrier()
    step_ms, exch_ms = max_over_ranks([e0.elapsed_time(e1) / K, x0.elapsed_time(x1) / K], dev)
    tokens = w.gpu_tokens
    return {"workload": "llama70b", "split": "token ranges on the chunk grid, older tokens on lower ranks",
            "ranks": R.world, "gpu_tokens_total": tokens, "tokens_this_rank": mine.gpu_tokens,
            "ms_per_step": step_ms, "kv_tokens_per_s": tokens / (step_ms * 1e-3),
            "exchange": "all-gather of B*Hq*(D+1) floats per rank into local memory, then hg_attn_merge over the ranks' rows",
            "exchange_bytes_per_rank": int(eng.record.numel() * 4), "exchange_ms": exch_ms,
            "exchange_share": exch_ms / step_ms if step_ms > 0 else None, "scaling": "strong"}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="all", help="one of tiny, opt13b, opt30b, llama70b, ragged; all (default); or handoff (the hand-off kernel alone)")
    ap.add_argument("--repeats", type=int, default=5, help="times the K-step pass is repeated per workload")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=0, help="keep only the first BATCH sequences (small profiling captures)")
    ap.add_argument("--chunk", type=int, default=0, help="override the workload's chunk_tokens (sweeps)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sharded", action="store_true", help="add the token-sharded record even on one rank")
    ap.add_argument("--probe", action="store_true", help="time the read-probe kernel for the launch-bound case too")
    ap.add_argument("--no-probe", action="store_true", help="skip the read-probe kernel")
    ap.add_argument("--extras", action="store_true",
                    help="also time the hand-off kernel, the host logits calculator and the residency operations")
    ap.add_argument("--launch-check", action="store_true",
                    help="only start the ranks (gloo, no GPU needed) and print which ranks met; not a bench line")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: start the ranks, one per GPU; rank 0's line is this command's line
        print(f"bench.py: starting {args.gpus} ranks through torch.distributed.run", file=sys.stderr, flush=True)
        raise SystemExit(subprocess.call(launcher_command(sys.argv[1:], args.gpus), cwd=ROOT))

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.launch_check:
        import torch.distributed as dist
        dist.init_process_group("gloo")
        seen = [None] * world
        dist.all_gather_object(seen, rank)
        got = max_over_ranks([float(rank)])
        dist.barrier()
        dist.destroy_process_group()
        if rank == 0:
            print(json.dumps({"launch_check": True, "world": world, "ranks_seen": seen, "max_rank": got[0]}), flush=True)
        return
    if args.impl == "reference":
        return run_reference(args, rank, world)

    import torch
    import torch.distributed as dist

    print(f"bench.py: rank {rank} of {world}", file=sys.stderr, flush=True)
    if not torch.cuda.is_available():
        raise SystemExit(f"bench.py (rank {rank} of {world}) needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    R = Ranks(rank, local_rank, world)
    if world > 1:
        os.environ.setdefault("NCCL_DEBUG", "INFO")          # communicator lines (ranks, transport) stay visible
        os.environ.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/dev/stderr")   # standard output carries the one JSON line only
        dist.init_process_group("nccl", device_id=torch.device(R.dev))

    # the group-query configurations first: their consumer warps are the most clock-sensitive, and the 7.5 GB
    # configuration leaves the board at its power cap for the measurements that follow it
    if args.workload == "handoff":              # only the hand-off kernel (profiling captures); not a bench line
        print(json.dumps({"handoff": time_handoff(R.dev, args.steps)}), flush=True)
        return
    names = ["tiny", "ragged", "llama70b", "opt13b", "opt30b"] if args.workload == "all" else [args.workload]
    head_name = HEADLINE if args.workload == "all" else args.workload
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.3)
    # (the hand-off kernel's two short measurements come first for the same reason)
    handoff = time_handoff(R.dev, args.steps) if args.workload == "all" and rank == 0 else None
    recs = {n: measure_workload(n, args, R, sampler) for n in names}
    shard_rec = measure_sharded(args, R) if (world > 1 or args.sharded) and args.workload == "all" else None
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    if rank != 0:
        return
    time.sleep(0.2)
    head = recs[head_name]
    hl = head.pop("_headline")
    for r in recs.values():
        r.pop("_headline", None)
    sampler.stop()
    config = {k: head[k] for k in ("workload", "batch", "q_heads", "kv_heads", "head_dim", "kv_dtype", "context", "gpu_tokens",
                                  "page_size", "chunk_tokens", "kv_bytes_per_step", "l2", "partial_us", "merge_us",
                                  "kernel_timing", "probe_us", "extras", "repeats_ms_per_step")}
    config["step_gbs"] = head.get("step_gbs")
    config["step_frac_of_8000"] = head.get("step_frac_of_8000")
    config["headline"] = f"the median of {max(1, args.repeats)} repeats of {args.steps} steps of `{head['workload']}`"
    if args.workload == "all":
        config["workloads"] = [recs[n] for n in names]
        config["min_step_frac_of_8000"] = min(recs[n]["step_frac_of_8000"] for n in LARGE)
        config["handoff"] = handoff
    line = {
        "metric": METRIC, "value": head["kv_tokens_per_s"], "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": hl["ms_step"], "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config, "roofline": head["roofline"], "e2e": head["e2e"],
        "gpu_launches": 2 * args.steps,
        "clocks": head["clocks"],
    }
    if shard_rec is not None:
        line["sharded"] = shard_rec
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = time_oracle(hl["w"], R.dev)[0]
    elif world == 1:
        line["cpu_baseline"] = None
    print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()

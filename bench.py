#!/usr/bin/env python
"""Benchmark of the hybrid decode-attention hot path on B200.

A step is one pass of the whole path over one batch of synthetic input: hg_attn_partial over the
GPU-resident KV slice, then hg_attn_merge of the chunk partials with the partials of the host-held
slice.  Prints ONE JSON line (rank 0).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

N > 1 is launched under torchrun, one rank per GPU; every rank runs its own copy of the workload
(independent sequences, no data-path collective): weak scaling.
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
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the partial kernel, from the ncu
# captures summarised under profiles/ (None until a capture of that workload exists)
NCU_TRAFFIC_BYTES = {
    # profiles/partial_kernel_opt13b.md: two sequences captured (805.55 MB read + 5.01 MB written), x 4
    "opt13b": 4 * (805_546_496 + 5_009_664),
    # profiles/partial_kernel_llama70b.md: the full launch captured
    "llama70b": 1_718_226_000 + 7_822_080,
    # profiles/partial_kernel_opt30b.md: one of the four sequences captured (1879.14 MB read + 3.87 MB written), x 4
    "opt30b": 4 * (1_879_144_000 + 3_870_464),
    # profiles/partial_kernel_ragged.md: the full launch captured
    "ragged": 951_494_144 + 8_356_864,
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


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "25"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            pass
        rows = [l for t, l in self.lines if t0 - 0.05 <= t <= t1 + 0.2] or [l for _, l in self.lines]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            p = [x.strip() for x in l.split(",")]
            try:
                sm.append(float(p[0])); mx.append(float(p[1]))
            except Exception:
                continue
            for n, v in zip(names, p[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


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
    return {"value": tokens / dt, "unit": UNIT, "cores": threads, "kind": "oracle",
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
    return out


def run_reference(args, rank, world):
    """--impl reference: the fp64 oracle on the host cores, each step a bounded sample of the workload."""
    if rank != 0:
        return
    import torch
    from oracle import hg_oracle as O
    from paper_2604_18529_b200 import workload as W
    w = W.make_workload(args.workload)
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
            "config": {"workload": args.workload, "sample": f"{len(items)} of {w.B * w.Hq} (sequence, head) rows per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle",
                             "sample": f"{len(items)} rows x {args.steps} steps"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--workload", default="opt13b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=0, help="keep only the first BATCH sequences (small profiling captures)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--probe", action="store_true", help="also time the read-probe kernel")
    ap.add_argument("--extras", action="store_true",
                    help="also time the hand-off kernel, the host logits calculator and the residency operations")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        return run_reference(args, rank, world)

    import torch
    import torch.distributed as dist
    import paper_2604_18529_b200 as pkg
    from paper_2604_18529_b200 import workload as W
    from paper_2604_18529_b200.problem import DeviceProblem

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    w = W.make_workload(args.workload)
    if args.batch:
        w = W.first_sequences(w, args.batch)
    prob = DeviceProblem(w, dev)
    # partials of the host-held slice: produced by the host in the real system; here synthetic values with
    # the statistics of a real partial (they are inputs of the merge, not results of this library)
    gen = torch.Generator(device=dev).manual_seed(w.seed)
    host = [(torch.randn(w.B, w.Hq, 1, w.D, device=dev, generator=gen),
             torch.randn(w.B, w.Hq, 1, device=dev, generator=gen),
             torch.rand(w.B, w.Hq, 1, device=dev, generator=gen) + 1.0)]
    stream = torch.cuda.current_stream()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step = prob.prepare_step(host)          # both calls with their arguments marshalled once, as a decode loop would
    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if int(prob.status.item()) != 0:
        raise SystemExit(f"device status {int(prob.status.item())} after warm-up")

    # ---- pass A: exactly K steps, device-timed ------------------------------------------------------
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    t_wall0 = time.time()
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms_total = ev0.elapsed_time(ev1)

    # ---- pass B: K more steps with an event around every kernel (roofline of the dominant kernel) --------
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    for e in evs:
        e[0].record(stream); prob.partial(); e[1].record(stream); prob.merge(host); e[2].record(stream)
    torch.cuda.synchronize()
    t_wall1 = time.time()
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    part_ms = [e[0].elapsed_time(e[1]) for e in evs]
    merge_ms = [e[1].elapsed_time(e[2]) for e in evs]

    # ---- end to end: per-step data in pinned host memory, results read back ----------------------------------
    pin = lambda t: t.cpu().pin_memory()
    q_h, sl_h, tb_h, te_h = pin(prob.q), pin(prob.seq_lens), pin(prob.tok_begin), pin(prob.tok_end)
    host_h = [tuple(pin(x) for x in src) for src in host]
    out_h = torch.empty(prob.out.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(prob.lse.shape, dtype=torch.float32).pin_memory()
    ws = torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, 1), dtype=torch.uint8, device=dev)

    decode_host = pkg.prepare_decode_host(q_h, prob.kv["k"], prob.kv["v"], sl_h, tb_h, te_h, host_h, out_h, lse_h, ws,
                                          prob.desc)     # arguments marshalled once, as a decode loop would

    def e2e_step():
        decode_host()
        stream.synchronize()            # the caller reads out_h / lse_h after every step

    for _ in range(3):
        e2e_step()
    barrier()
    ee0, ee1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ee0.record(stream)
    for _ in range(args.steps):
        e2e_step()
    ee1.record(stream)
    barrier()
    e2e_ms = ee0.elapsed_time(ee1)
    same = torch.equal(out_h, prob.out.cpu()) and torch.equal(lse_h, prob.lse.cpu())
    h2d = sum(t.numel() * t.element_size() for t in (q_h, sl_h, tb_h, te_h)) + \
        sum(t.numel() * t.element_size() for src in host_h for t in src)
    d2h = out_h.numel() * 4 + lse_h.numel() * 4

    probe_ms = None
    if args.probe:
        sink = torch.zeros(w.B, w.Hkv, prob.NC, dtype=torch.int32, device=dev)
        pe = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(args.steps)]
        for _ in range(3):
            pkg.hg_kv_read_probe(prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, sink, prob.desc)
        for e in pe:
            e[0].record(stream)
            pkg.hg_kv_read_probe(prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, sink, prob.desc)
            e[1].record(stream)
        torch.cuda.synchronize()
        probe_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in pe)

    extras = time_extras(w, prob, dev, args.steps) if args.extras and rank == 0 else None
    ms_total, e2e_ms = max_over_ranks([ms_total, e2e_ms], dev)

    if rank == 0:
        tokens = w.gpu_tokens
        ms_step = ms_total / args.steps
        peak, peak_kind = measured_peak()
        kv_bytes = w.kv_bytes()
        nchunks = sum(w.chunk_grid(b)[1] for b in range(w.B))
        part_alg = kv_bytes + w.B * w.Hq * w.D * 2 + (prob.kv["num_pages"] * 4 if w.paged else 0) + \
            w.Hq * nchunks * (w.D + 2) * 4
        part_avg = statistics.mean(part_ms)
        achieved = part_alg / (part_avg * 1e-3) / 1e9
        line = {
            "metric": METRIC, "value": whole_job_value(tokens, world, ms_step), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": w.name, "batch": w.B, "q_heads": w.Hq, "kv_heads": w.Hkv, "head_dim": w.D,
                       "kv_dtype": w.dtype, "context": max(w.seq_lens), "gpu_tokens": tokens, "page_size": w.page_size,
                       "chunk_tokens": w.chunk_tokens, "kv_bytes_per_step": kv_bytes,
                       "l2": "inputs larger than L2" if kv_bytes > 2 * 126e6 else "inputs fit L2 (launch-bound case)",
                       "step_gbs": prob.alg_bytes() / (ms_step * 1e-3) / 1e9,
                       "step_frac_of_8000": prob.alg_bytes() / (ms_step * 1e-3) / 1e9 / 8000.0,
                       "partial_us": part_avg * 1e3, "merge_us": statistics.mean(merge_ms) * 1e3,
                       "roofline_timing": "second pass of K steps with CUDA events around each kernel",
                       "probe_us": None if probe_ms is None else probe_ms * 1e3, "extras": extras},
            "roofline": {"bound": "hbm", "kernel": "partial_kernel", "achieved": achieved, "peak": peak,
                         "peak_kind": f"{peak_kind} copy bandwidth", "unit": "GB/s", "frac": achieved / peak,
                         "frac_of_8000": achieved / 8000.0, "alg_bytes_per_launch": part_alg,
                         "traffic": None if args.batch else NCU_TRAFFIC_BYTES.get(args.workload)},
            "e2e": {"value": whole_job_value(tokens, world, e2e_ms / args.steps), "unit": UNIT, "h2d_bytes_per_step": h2d,
                    "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.steps, "matches_device_path": bool(same),
                    "api": "hg_attn_decode_host via prepare_decode_host (KV pools stay device resident: they are the GPU's slice of the cache)"},
            "gpu_launches": 2 * args.steps,
            "clocks": clocks,
        }
        if not args.no_cpu_baseline and world == 1:
            line["cpu_baseline"] = time_oracle(w, dev)[0]
        elif world == 1:
            line["cpu_baseline"] = None
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

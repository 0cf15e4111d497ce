"""Token-range sharding over several ranks, checked without a GPU: the split plan, the identity that
lets a merged row travel as a partial, and the exchange itself on two gloo ranks with the oracle
standing in for each rank's local decode."""
import os
import random
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import hg_oracle as O
from paper_2604_18529_b200 import sharded
from paper_2604_18529_b200.workload import make_workload

from parity_util import bits

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("world", [1, 2, 3, 4, 8])
def test_shard_ranges_tile_the_slice_on_the_chunk_grid(world):
    rng = random.Random(world)
    for chunk in (64, 256, 2048):
        tb = [0, 5, 13108, 4096, 700, 9000]
        te = [0, 5, 32768, 4096 + 2 * chunk, 701, 9000 + rng.randrange(1, 40000)]
        begins, ends = sharded.shard_ranges(tb, te, world, chunk)
        assert len(begins) == len(ends) == world
        for b in range(len(tb)):
            pos = tb[b]
            sizes = []
            for r in range(world):
                lo, hi = begins[r][b], ends[r][b]
                assert lo <= hi
                if hi > lo:
                    assert lo == pos                           # consecutive, older tokens on lower ranks
                    assert lo == tb[b] or lo % chunk == 0      # cuts only on the absolute chunk grid
                    assert hi == te[b] or hi % chunk == 0
                    pos = hi
                    sizes.append(-(-hi // chunk) - lo // chunk)
            assert pos == te[b]                                # nothing lost, nothing twice
            if sizes and len(sizes) == world:
                assert max(sizes) - min(sizes) <= 1            # chunks dealt evenly


def test_shard_ranges_rejects_bad_input():
    with pytest.raises(ValueError):
        sharded.shard_ranges([0], [10], 0, 64)
    with pytest.raises(ValueError):
        sharded.shard_ranges([10], [5], 2, 64)


def test_merged_row_is_a_partial_with_unit_sum():
    """(out, lse, 1) of each token range, merged, is attention over the union (Section 4.2's exactness
    claim applied twice) - including ranges that are empty."""
    rng = np.random.default_rng(7)
    D, L = 8, 97
    q = rng.standard_normal(D).astype(np.float16).view(np.uint16)
    K = rng.standard_normal((L, D)).astype(np.float16).view(np.uint16)
    V = rng.standard_normal((L, D)).astype(np.float16).view(np.uint16)
    ref_out, ref_lse = O.full(q, K, V, "f16")
    for cuts in ([0, 40, 97], [0, 0, 33, 33, 97], [0, 1, 2, 96, 97], [0, 97, 97]):
        m, l, o = [], [], []
        for lo, hi in zip(cuts[:-1], cuts[1:]):
            if hi == lo:
                out_r, lse_r = np.zeros(D), -np.inf
            else:
                out_r, lse_r = O.full(q, K, V, "f16", t0=lo, n=hi - lo)
            m.append(lse_r); l.append(1.0); o.append(out_r)
        out, lse = O.merge(np.array(m), np.array(l), np.array(o))
        assert np.abs(out - ref_out).max() < 1e-13 and abs(lse - ref_lse) < 1e-13


def test_record_layout_round_trip():
    B, Hq, D = 3, 5, 64
    out = torch.arange(B * Hq * D, dtype=torch.float32).view(B, Hq, D)
    lse = -torch.arange(B * Hq, dtype=torch.float32).view(B, Hq)
    rec = sharded.pack_record(out, lse)
    assert rec.numel() == sharded.record_floats(B, Hq, D) and rec.numel() % sharded.RECORD_ALIGN == 0
    gathered = torch.stack([rec, 2 * rec])
    srcs = sharded.record_sources(gathered, B, Hq, D)
    assert len(srcs) == 2
    o0, m0, l0 = srcs[0]
    o1, m1, _ = srcs[1]
    assert o0.shape == (B, Hq, 1, D) and m0.shape == (B, Hq, 1) and l0.shape == (B, Hq, 1)
    assert torch.equal(o0[:, :, 0], out) and torch.equal(m0[:, :, 0], lse) and (l0 == 1).all()
    assert torch.equal(o1[:, :, 0], 2 * out) and torch.equal(m1[:, :, 0], 2 * lse)
    assert o0.is_contiguous() and m0.is_contiguous()          # the merge kernel reads them as dense arrays
    for t in (o1, m0, m1):                                    # every block starts 256 bytes apart at least
        assert (t.data_ptr() - gathered.data_ptr()) % 256 == 0


def _rank(rank, world, port, q):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = make_workload("tiny")
        qb, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
        begins, ends = sharded.shard_ranges(w.tok_begin, w.tok_end, world, w.chunk_tokens)
        # this rank's local decode, by the oracle: attention over its own token range
        out_r, lse_r = O.full_batch(qb, K, V, w.dtype, begins[rank], ends[rank])
        rec = sharded.pack_record(torch.from_numpy(out_r).float(), torch.from_numpy(lse_r).float())
        gathered = sharded.exchange_records(rec)
        srcs = sharded.record_sources(gathered, w.B, w.Hq, w.D)
        o = np.stack([s[0][:, :, 0].double().numpy() for s in srcs], axis=2)       # [B][Hq][world][D]
        m = np.stack([s[1][:, :, 0].double().numpy() for s in srcs], axis=2)
        l = np.stack([s[2][:, :, 0].double().numpy() for s in srcs], axis=2)
        out, lse = O.merge_batch(m, l, o)
        ref_out, ref_lse = O.full_batch(qb, K, V, w.dtype, w.tok_begin, w.tok_end)
        q.put((rank, float(np.abs(out - ref_out).max()), float(np.abs(lse - ref_lse).max()),
               [int(e - b) for b, e in zip(begins[rank], ends[rank])]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_exchange_and_merge_on_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=180) for _ in range(2))
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    w = make_workload("tiny")
    assert sum(sum(g[3]) for g in got) == w.gpu_tokens            # the two ranks covered the slice between them
    assert all(sum(g[3]) > 0 for g in got)
    for _, out_err, lse_err, _ in got:                            # every rank ends with the full result
        assert out_err < 2e-6 and lse_err < 2e-6                  # the record travels as fp32

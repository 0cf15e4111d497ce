"""Token-sharded decode on the GPU against the oracle.

One GPU is available, so the ranks of a world are run one after another on it (each over its own token
range of the same pool: a rank never reads outside its range) and their records are placed in the
gathered buffer where the all-gather would land them; the combine is the library's merge.  The
collective itself runs here on a one-rank NCCL group, and on two gloo ranks in the CPU tests.
"""
import os

import numpy as np
import pytest
import torch
import torch.distributed as dist

from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import sharded
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import OracleRef, check_output

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _i32(x):
    return torch.tensor(x, dtype=torch.int32, device=DEV)


def sharded_result(prob, ref, world, host_on_rank=0):
    """Run ``world`` emulated ranks in turn and merge their records; returns (out, lse, tokens per rank)."""
    w = prob.w
    begins, ends = sharded.shard_ranges(w.tok_begin, w.tok_end, world, w.chunk_tokens)
    n = sharded.record_floats(w.B, w.Hq, w.D)
    gathered = torch.full((world, n), float("nan"), dtype=torch.float32, device=DEV)
    host = ref.host_partials_device(DEV)
    ws = torch.empty(hg.hg_attn_workspace_bytes(prob.desc, len(host)), dtype=torch.uint8, device=DEV)
    for r in range(world):
        rec = gathered[r]
        out_r = rec[:w.B * w.Hq * w.D].view(w.B, w.Hq, w.D)
        lse_r = rec[w.B * w.Hq * w.D:w.B * w.Hq * (w.D + 1)].view(w.B, w.Hq)
        hg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, _i32(begins[r]), _i32(ends[r]),
                          host if r == host_on_rank else [], out_r, lse_r, ws, prob.desc)
    out = torch.empty(w.B, w.Hq, w.D, dtype=torch.float32, device=DEV)
    lse = torch.empty(w.B, w.Hq, dtype=torch.float32, device=DEV)
    hg.hg_attn_merge(sharded.record_sources(gathered, w.B, w.Hq, w.D), out, lse, prob.desc)
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    return out, lse, [sum(e - b for b, e in zip(begins[r], ends[r])) for r in range(world)]


@pytest.mark.parametrize("name", ["opt13b", "llama70b", "ragged"])
@pytest.mark.parametrize("world", [2, 4, 8])
def test_token_sharded_equals_monolithic_attention(name, world):
    full = W.make_workload(name)
    w = W.scaled_down(full, 64 if name != "ragged" else 16, max_batch=3)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    out, lse, per_rank = sharded_result(prob, ref, world, host_on_rank=world - 1)
    assert sum(per_rank) == w.gpu_tokens
    check_output(out, lse, ref.out, ref.lse, f"{name} over {world} ranks")
    # and against the same problem on one device: same real-valued result, other summation order
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    bound = 1e-5 * max(1.0, prob.out.abs().max().item())
    assert (out - prob.out).abs().max().item() < bound and (lse - prob.lse).abs().max().item() < 1e-5


def test_ranks_with_nothing_to_do_contribute_nothing():
    # three chunks, eight ranks: five ranks hold no token at all; the second sequence's slice is empty
    w = W.AttnWorkload(name="few", B=2, Hq=8, Hkv=2, D=128, dtype="bf16", seq_lens=[600, 300], tok_begin=[100, 40],
                       tok_end=[333, 40], page_size=16, layout="HND", chunk_tokens=128, seed=5)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    out, lse, per_rank = sharded_result(prob, ref, 8)
    assert sorted(per_rank)[:5] == [0] * 5
    check_output(out, lse, ref.out, ref.lse, "idle ranks")


@pytest.fixture
def one_rank_nccl():
    if dist.is_initialized():
        pytest.skip("a process group is already up")
    port = 33500 + os.getpid() % 2000
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                            device_id=torch.device(DEV))
    try:
        yield
    finally:
        dist.destroy_process_group()


def test_step_through_a_one_rank_nccl_group(one_rank_nccl):
    w = W.scaled_down(W.make_workload("llama70b"), 64)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    eng = sharded.TokenShardedDecode(prob.desc, device=DEV)
    assert eng.world == 1
    out = torch.empty_like(prob.out)
    lse = torch.empty_like(prob.lse)
    with torch.cuda.device(DEV):
        for _ in range(2):                                     # buffers are reused from step to step
            eng.step(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                     ref.host_partials_device(DEV), out, lse)
        torch.cuda.synchronize()
    check_output(out, lse, ref.out, ref.lse, "one-rank group")
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    assert (out - prob.out).abs().max().item() < 1e-6
    assert np.isfinite(eng.gathered.cpu().numpy()).all()

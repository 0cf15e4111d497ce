"""The allocation-free decode entry point (collected last on purpose).

Some callers cannot call cudaMalloc: code running inside a CUDA-graph capture, plugins that get a
fixed memory budget from their host application, decode loops that must never touch the allocator.
``hg_attn_decode_static`` serves them by keeping the chunk partials in a fixed array inside the
library.  It must give what ``hg_attn_decode`` gives with a caller workspace, also on a second call
that finds the previous call's data still in the array, and it must refuse problems whose partials
exceed the array."""
import pytest
import torch

import paper_2604_18529_b200 as pkg
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import OUT_MAX_ABS, LSE_ABS

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def both_ways(w):
    prob = DeviceProblem(w, DEV)
    gen = torch.Generator(device=DEV).manual_seed(w.seed)
    host = [(torch.randn(w.B, w.Hq, 1, w.D, device=DEV, generator=gen),
             torch.randn(w.B, w.Hq, 1, device=DEV, generator=gen),
             torch.rand(w.B, w.Hq, 1, device=DEV, generator=gen) + 1.0)]
    ws = torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, 1), dtype=torch.uint8, device=DEV)
    want_out, want_lse = torch.empty_like(prob.out), torch.empty_like(prob.lse)
    pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, host,
                       want_out, want_lse, ws, prob.desc)
    out = torch.full_like(prob.out, float("nan")); lse = torch.full_like(prob.lse, float("nan"))
    before = torch.cuda.memory_allocated()
    pkg.hg_attn_decode_static(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, host,
                              out, lse, prob.desc)
    assert torch.cuda.memory_allocated() == before
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    assert (out - want_out).abs().max().item() <= OUT_MAX_ABS
    assert (lse - want_lse).abs().max().item() <= LSE_ABS
    return out


def test_static_scratch_decode_matches_workspace_decode_twice_in_a_row():
    big = W.AttnWorkload("first", 2, 8, 2, 128, "f16", [3000, 1111], [500, 64], [3000, 1000], page_size=16,
                         chunk_tokens=256, seed=31)
    small = W.AttnWorkload("second", 1, 4, 4, 64, "bf16", [700], [130], [650], page_size=32, layout="NHD",
                           chunk_tokens=128, seed=32)
    both_ways(big)      # leaves its partials in the shared array
    both_ways(small)    # a different shape over the stale contents
    both_ways(big)


def test_static_scratch_decode_refuses_problems_beyond_its_limit():
    # 64 heads x 1100 chunks x 130 floats x 4 bytes > 8 MiB: refused before anything is launched
    w = W.AttnWorkload("too_big", 1, 64, 8, 128, "f16", [70400], [0], [70400], page_size=16, chunk_tokens=64, seed=33)
    prob = DeviceProblem(w, DEV)
    need = w.B * w.Hq * prob.NC * (w.D + 2) * 4
    assert need > hg.HG_STATIC_SCRATCH_BYTES
    with pytest.raises(hg.HgError) as e:
        pkg.hg_attn_decode_static(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, [],
                                  prob.out, prob.lse, prob.desc)
    assert e.value.status == hg.HG_ERR_WORKSPACE

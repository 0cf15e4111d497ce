"""The allocation-free decode entry point (collected last on purpose).

Some callers cannot call cudaMalloc: plugins that get a fixed memory budget from their host application,
decode loops that must never touch the allocator, components that are handed their buffers and own none.
``hg_attn_decode_static`` serves them by keeping the chunk partials in a fixed array inside the
library.  It runs the kernels ``hg_attn_decode`` runs, in the same order, so it must give the same bits -
also on a second call that finds the previous call's data still in the array - and those bits must match
the oracle; a call must leave the device's free memory as it found it; and it must accept a problem whose
partials fill the array exactly and refuse one that exceeds it."""
import pytest
import torch

import paper_2604_18529_b200 as pkg
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import OracleRef, check_output

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def both_ways(w, oracle=True):
    prob = DeviceProblem(w, DEV)
    if oracle:
        ref = OracleRef(w)
        host = ref.host_partials_device(DEV)
    else:
        host = []
    ws = torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, len(host)), dtype=torch.uint8, device=DEV)
    want_out, want_lse = torch.empty_like(prob.out), torch.empty_like(prob.lse)
    pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, host,
                       want_out, want_lse, ws, prob.desc)
    out = torch.full_like(prob.out, float("nan")); lse = torch.full_like(prob.lse, float("nan"))
    args = (prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, host, out, lse, prob.desc)
    pkg.hg_attn_decode_static(*args)             # (the first call on a device also looks the array's address up)
    torch.cuda.synchronize()
    first = (out.clone(), lse.clone())
    # a further call must not change what the driver reports as free device memory: cudaMemGetInfo sees every
    # allocation of the process, not only those of torch's caching allocator
    free_before, _ = torch.cuda.mem_get_info()
    torch_before = torch.cuda.memory_allocated()
    out.fill_(float("nan")); lse.fill_(float("nan"))
    pkg.hg_attn_decode_static(*args)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before and torch.cuda.memory_allocated() == torch_before
    assert int(prob.status.item()) == hg.HG_DEV_OK
    for o, l in (first, (out, lse)):
        assert torch.equal(o, want_out) and torch.equal(l, want_lse)          # same kernels, same order: same bits
    if oracle:
        check_output(out, lse, ref.out, ref.lse, w.name)
    return out


def test_static_scratch_decode_matches_workspace_decode_and_the_oracle_twice_in_a_row():
    big = W.AttnWorkload("first", 2, 8, 2, 128, "f16", [3000, 1111], [500, 64], [3000, 1000], page_size=16,
                         chunk_tokens=256, seed=31)
    small = W.AttnWorkload("second", 1, 4, 4, 64, "bf16", [700], [130], [650], page_size=32, layout="NHD",
                           chunk_tokens=128, seed=32)
    both_ways(big)      # leaves its partials in the shared array
    both_ways(small)    # a different shape over the stale contents
    both_ways(big)


def test_static_scratch_decode_accepts_partials_that_fill_the_array_exactly():
    # n = 57 heads x 283 chunks = 16131 partials: 512 n bytes of o plus twice 4 n bytes rounded up to 256 = 8 MiB exactly
    w = W.AttnWorkload("brim", 1, 57, 57, 128, "f16", [283 * 64], [0], [283 * 64], page_size=16, chunk_tokens=64, seed=34)
    n = w.B * w.Hq * w.num_chunks
    up = lambda x: -(-x // 256) * 256
    assert n == 16131 and up(n * 128 * 4) + 2 * up(n * 4) == hg.HG_STATIC_SCRATCH_BYTES
    both_ways(w, oracle=False)


def test_static_scratch_decode_refuses_problems_beyond_its_limit():
    # 64 heads x 1100 chunks x 130 floats x 4 bytes > 8 MiB: refused before anything is launched; so is one chunk
    # more than the problem that fills the array exactly
    brim = W.AttnWorkload("over", 1, 57, 57, 128, "f16", [284 * 64], [0], [284 * 64], page_size=16, chunk_tokens=64, seed=35)
    pb = DeviceProblem(brim, DEV)
    with pytest.raises(hg.HgError) as e:
        pkg.hg_attn_decode_static(pb.q, pb.kv["k"], pb.kv["v"], pb.seq_lens, pb.tok_begin, pb.tok_end, [], pb.out, pb.lse,
                                  pb.desc)
    assert e.value.status == hg.HG_ERR_WORKSPACE
    del pb
    w = W.AttnWorkload("too_big", 1, 64, 8, 128, "f16", [70400], [0], [70400], page_size=16, chunk_tokens=64, seed=33)
    prob = DeviceProblem(w, DEV)
    need = w.B * w.Hq * prob.NC * (w.D + 2) * 4
    assert need > hg.HG_STATIC_SCRATCH_BYTES
    with pytest.raises(hg.HgError) as e:
        pkg.hg_attn_decode_static(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, [],
                                  prob.out, prob.lse, prob.desc)
    assert e.value.status == hg.HG_ERR_WORKSPACE

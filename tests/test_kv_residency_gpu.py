"""KV residency on the GPU: appending each step's K/V rows, attending over the grown slice, then evicting the
oldest tokens to the host and attending over the shrunk slice.  Data movement is checked bit for bit against
the logical rows of the workload generator, attention against the oracle."""
import dataclasses

import numpy as np

import pytest
import torch

import paper_2604_18529_b200 as pkg
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import OracleRef, check_output

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
STEPS = 5


def rows_at(w, which, t_by_seq):
    """[B][Hkv][D] rows of token t_by_seq[b]."""
    return torch.stack([torch.stack([w.kv_rows(which, b, g, t, t + 1)[0] for g in range(w.Hkv)])
                        for b, t in enumerate(t_by_seq)]).to(DEV)


def poison_future_rows(prob, w, first_t):
    """Rows at positions >= first_t[b] of resident pages get NaN patterns: only hg_kv_append may bring them to life."""
    kv, ps = prob.kv, w.page_size
    hnd = w.paged and w.layout == "HND"
    for b in range(w.B):
        for t in range(first_t[b], w.seq_lens[b]):
            pg = t // ps
            phys = int(kv["block_table"][b, pg]) if w.paged else b * kv["max_pages"] + pg
            for pool in (kv["k"], kv["v"]):
                if hnd:
                    pool[phys, :, t % ps, :] = float("nan")
                else:
                    pool[phys, t % ps, :, :] = float("nan")


@pytest.mark.parametrize("layout,paged", [("HND", True), ("NHD", True), ("NHD", False)])
@pytest.mark.parametrize("G", [1, 4])
def test_append_then_attend_then_evict_then_attend(layout, paged, G):
    final = W.AttnWorkload("life", 2, 2 * G, 2, 128, "f16", [700, 411], [130, 40], [700, 411], page_size=16, layout=layout,
                           paged=paged, chunk_tokens=128, seed=90 + G)
    start = [L - STEPS for L in final.seq_lens]
    prob = DeviceProblem(final, DEV)                    # pool and block table sized for the final lengths
    poison_future_rows(prob, final, start)
    prob.seq_lens = torch.tensor(start, dtype=torch.int32, device=DEV)
    prob.tok_end = torch.tensor(start, dtype=torch.int32, device=DEV)

    # ---- decode steps: append the new token's K, V, then attend (Section 2.1) ----
    for k in range(STEPS):
        t_new = [s + k for s in start]
        pkg.hg_kv_append(rows_at(final, "k", t_new), rows_at(final, "v", t_new), prob.kv["k"], prob.kv["v"],
                         prob.seq_lens, prob.tok_end, prob.desc)
        now = dataclasses.replace(final, seq_lens=[t + 1 for t in t_new], tok_end=[t + 1 for t in t_new])
        assert prob.seq_lens.tolist() == now.seq_lens and prob.tok_end.tolist() == now.tok_end
        ref = OracleRef(now)
        prob.step(ref.host_partials_device(DEV))
        torch.cuda.synchronize()
        assert int(prob.status.item()) == hg.HG_DEV_OK
        check_output(prob.out, prob.lse, ref.out, ref.lse, f"after append {k}")

    # ---- eviction: the oldest tokens of each slice leave for the host ----
    n_evict = [100, 37]
    max_evict, max_freed = 128, 16
    k_out = torch.full((final.B, max_evict, final.Hkv, final.D), 9.0, dtype=torch.float16, device=DEV)
    v_out = torch.full_like(k_out, 9.0)
    freed = torch.full((final.B, max_freed), 77, dtype=torch.int32, device=DEV)
    n_freed = torch.zeros(final.B, dtype=torch.int32, device=DEV)
    table_before = None if not paged else prob.kv["block_table"].clone()
    pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, torch.tensor(n_evict, dtype=torch.int32, device=DEV),
                    k_out, v_out, freed, n_freed, prob.desc)
    torch.cuda.synchronize()
    new_begin = [tb + ne for tb, ne in zip(final.tok_begin, n_evict)]
    assert prob.tok_begin.tolist() == new_begin
    ps = final.page_size
    for b in range(final.B):
        for g in range(final.Hkv):
            for which, out in (("k", k_out), ("v", v_out)):
                want = final.kv_rows(which, b, g, final.tok_begin[b], new_begin[b])
                assert torch.equal(out[b, : n_evict[b], g].cpu(), want)
        gone = list(range(final.tok_begin[b] // ps, new_begin[b] // ps))       # pages wholly below the new beginning
        if paged:
            assert (prob.kv["block_table"][b, gone] == -1).all()
            assert n_freed[b].item() == len(gone)
            assert freed[b, : len(gone)].tolist() == table_before[b, gone].tolist() and (freed[b, len(gone):] == -1).all()
            keep = [p for p in range(new_begin[b] // ps, -(-final.seq_lens[b] // ps))]
            assert torch.equal(prob.kv["block_table"][b, keep], table_before[b, keep])
        else:
            assert n_freed[b].item() == 0
    # the evicted rows are what the host-side logits calculator reads: attend over the shrunk slice
    after = dataclasses.replace(final, tok_begin=new_begin)
    ref = OracleRef(after)
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    check_output(prob.out, prob.lse, ref.out, ref.lse, "after eviction")


def test_evicting_more_than_the_slice_empties_it_and_append_needs_a_mapped_page():
    w = W.AttnWorkload("edge", 1, 2, 2, 64, "bf16", [100], [20], [100], page_size=16, chunk_tokens=64, seed=5)
    prob = DeviceProblem(w, DEV)
    k_out = torch.zeros(1, 256, 2, 64, dtype=torch.bfloat16, device=DEV); v_out = torch.zeros_like(k_out)
    pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, torch.tensor([1000], dtype=torch.int32, device=DEV),
                    k_out, v_out, None, None, prob.desc)
    torch.cuda.synchronize()
    assert prob.tok_begin.tolist() == [100]
    assert torch.equal(k_out[0, :80, 1].cpu(), w.kv_rows("k", 0, 1, 20, 100))
    prob.partial(); prob.merge([])
    torch.cuda.synchronize()
    assert (prob.out == 0).all() and torch.isinf(prob.lse).all()
    # position 100 lies on page 6, which holds tokens 96..111 and is still mapped: the append lands
    new = torch.ones(1, 2, 64, dtype=torch.bfloat16, device=DEV)
    pkg.hg_kv_append(new, new, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_end, prob.desc)
    torch.cuda.synchronize()
    assert prob.seq_lens.tolist() == [101] and prob.tok_end.tolist() == [101] and int(prob.status.item()) == 0
    # fill the page; position 112 needs page 7, which was never allocated: the row is dropped and reported
    for _ in range(11):
        pkg.hg_kv_append(new, new, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_end, prob.desc)
    torch.cuda.synchronize()
    assert prob.seq_lens.tolist() == [112] and int(prob.status.item()) == 0
    pkg.hg_kv_append(new, new, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_end, prob.desc)
    torch.cuda.synchronize()
    assert prob.seq_lens.tolist() == [112] and int(prob.status.item()) == hg.HG_DEV_BAD_PAGE


def test_a_full_freed_list_stops_the_eviction_instead_of_losing_pages():
    """Two pages fit the freed list, the request would empty five: the sequence keeps the pages that cannot be
    reported, its slice then begins at the first of them, and a later call finishes the job."""
    w = W.AttnWorkload("freed", 2, 2, 2, 64, "f16", [400, 300], [37, 10], [400, 300], page_size=16, chunk_tokens=64, seed=7)
    prob = DeviceProblem(w, DEV)
    table0 = prob.kv["block_table"].clone()
    max_evict, max_freed = 128, 2
    k_out = torch.zeros(2, max_evict, 2, 64, dtype=torch.float16, device=DEV); v_out = torch.zeros_like(k_out)
    freed = torch.full((2, max_freed), 77, dtype=torch.int32, device=DEV)
    n_freed = torch.zeros(2, dtype=torch.int32, device=DEV)
    ne = torch.tensor([90, 20], dtype=torch.int32, device=DEV)
    pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, ne, k_out, v_out, freed, n_freed, prob.desc)
    torch.cuda.synchronize()
    # sequence 0: [37, 127) would empty pages 2..6 (five); pages 2 and 3 are listed, page 4 cannot be: begin = 64
    # sequence 1: [10, 30) empties page 0 only (page 1 still holds tokens 30, 31)
    assert prob.tok_begin.tolist() == [64, 30] and n_freed.tolist() == [2, 1]
    assert freed[0].tolist() == table0[0, 2:4].tolist() and freed[1].tolist() == [int(table0[1, 0]), -1]
    assert (prob.kv["block_table"][0, 2:4] == -1).all() and torch.equal(prob.kv["block_table"][0, 4:], table0[0, 4:])
    assert torch.equal(k_out[0, :27, 1].cpu(), w.kv_rows("k", 0, 1, 37, 64))        # the rows that did leave
    assert int(prob.status.item()) == hg.HG_DEV_OK
    # the rest of the request in a second call
    pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, torch.tensor([63, 0], dtype=torch.int32, device=DEV),
                    k_out, v_out, freed, n_freed, prob.desc)
    torch.cuda.synchronize()
    assert prob.tok_begin.tolist() == [96, 30] and n_freed.tolist() == [2, 0]      # pages 4, 5 listed; page 6 still cannot be
    after = dataclasses.replace(w, tok_begin=[96, 30])
    ref = OracleRef(after)
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    check_output(prob.out, prob.lse, ref.out, ref.lse, "after two truncated evictions")


def test_eviction_over_an_unmapped_page_leaves_the_sequence_alone():
    w = W.AttnWorkload("hole", 2, 2, 2, 64, "f16", [400, 300], [32, 16], [400, 300], page_size=16, chunk_tokens=64, seed=8)
    prob = DeviceProblem(w, DEV)
    prob.kv["block_table"][0, 3] = -1                      # a hole inside sequence 0's oldest tokens
    table0 = prob.kv["block_table"].clone()
    k_out = torch.zeros(2, 64, 2, 64, dtype=torch.float16, device=DEV); v_out = torch.zeros_like(k_out)
    freed = torch.full((2, 8), 77, dtype=torch.int32, device=DEV); n_freed = torch.zeros(2, dtype=torch.int32, device=DEV)
    pkg.hg_kv_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, torch.tensor([48, 48], dtype=torch.int32, device=DEV),
                    k_out, v_out, freed, n_freed, prob.desc)
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_BAD_PAGE
    assert prob.tok_begin.tolist() == [32, 64] and n_freed.tolist() == [0, 3]
    assert torch.equal(prob.kv["block_table"][0], table0[0]) and (freed[0] == -1).all()
    assert torch.equal(k_out[1, :48, 0].cpu(), w.kv_rows("k", 1, 0, 16, 64))


@pytest.mark.parametrize("G", [1, 4])
def test_eviction_beside_attention_gives_the_bits_of_the_serial_order(G):
    """The three-step eviction (begin on the attention's stream; row copy, device -> host copies and un-mapping on a
    second stream) with the attention of the same step running meanwhile over the shrunk slice: block table, freed
    list, host rows and attention output are bit for bit those of evicting first and attending afterwards, and the
    attention - merged with a host partial recomputed from the rows that arrived on the host - equals monolithic
    attention over the whole sequence."""
    from oracle import hg_oracle as O
    from paper_2604_18529_b200.hybrid import HostKvStore
    from parity_util import bits
    w = W.AttnWorkload("beside", 3, 2 * G, 2, 128, "f16", [3000, 1500, 900], [700, 100, 333], [3000, 1500, 900], page_size=16,
                       chunk_tokens=256, seed=60 + G)
    n_evict = [640, 333, 0]
    new_begin = [tb + ne for tb, ne in zip(w.tok_begin, n_evict)]
    after = dataclasses.replace(w, tok_begin=new_begin)
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    ref_out, ref_lse = O.full_batch(q, K, V, w.dtype, [0] * w.B, w.seq_lens)

    results = []
    for beside in (False, True):
        prob = DeviceProblem(w, DEV)
        # the host tier already holds the tokens below the old beginning
        store = HostKvStore(w.B, 2048, w.Hkv, w.D, torch.float16)
        for b in range(w.B):
            for g in range(w.Hkv):
                store.k[b, : w.tok_begin[b], g] = w.kv_rows("k", b, g, 0, w.tok_begin[b])
                store.v[b, : w.tok_begin[b], g] = w.kv_rows("v", b, g, 0, w.tok_begin[b])
            store.n[b] = w.tok_begin[b]
        freed = torch.full((w.B, 64), 77, dtype=torch.int32, device=DEV)
        n_freed = torch.zeros(w.B, dtype=torch.int32, device=DEV)
        # attention of the shrunk slice, with no host source: its partials must not depend on the order either
        if beside:
            pending = store.begin_evict(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, n_evict, prob.desc, freed, n_freed)
            prob.step([])                                  # enqueued right behind step 1, runs while the rows drain
            assert pending.wait() == n_evict
        else:
            store.evict_from_gpu(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, n_evict, prob.desc, freed, n_freed)
            prob.step([])
        torch.cuda.synchronize()
        assert int(prob.status.item()) == hg.HG_DEV_OK and prob.tok_begin.tolist() == new_begin
        assert store.n.tolist() == new_begin
        results.append((prob.out.clone(), prob.lse.clone(), prob.o_part.clone(), prob.kv["block_table"].clone(), freed.clone(),
                        n_freed.clone(), store.k.clone(), store.v.clone()))
        # the host rows are the sequence's prefix, bit for bit; the host partial comes from them
        hm = np.empty((w.B, w.Hq, 1)); hl = np.empty((w.B, w.Hq, 1)); ho = np.empty((w.B, w.Hq, 1, w.D))
        for b in range(w.B):
            for g in range(w.Hkv):
                assert torch.equal(store.k[b, : new_begin[b], g], w.kv_rows("k", b, g, 0, new_begin[b]))
                assert torch.equal(store.v[b, : new_begin[b], g], w.kv_rows("v", b, g, 0, new_begin[b]))
            for h in range(w.Hq):
                g = h // w.G
                hm[b, h, 0], hl[b, h, 0], ho[b, h, 0] = O.partial(q[b, h], bits(store.k[b, :, g]), bits(store.v[b, :, g]),
                                                                   w.dtype, t0=0, n=new_begin[b])
        prob.merge([tuple(torch.from_numpy(x).float().to(DEV) for x in (ho, hm, hl))])
        torch.cuda.synchronize()
        check_output(prob.out, prob.lse, ref_out, ref_lse, "beside" if beside else "serial")
    for a, b in zip(*results):
        assert torch.equal(a, b)
    assert (results[0][5] > 0).any()                       # pages did get freed and listed

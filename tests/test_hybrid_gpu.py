"""The whole hybrid step (GPU slice + CPU-selected host tokens, Algorithm 1 in the loop) against the oracle.

Every step's output must equal monolithic attention over exactly the tokens that took part in it - the GPU
slice plus the host tokens the CPU stage chose in that step - and the (K, strategy) sequence must be what
Algorithm 1 gives on the latencies the steps measured.
"""
import numpy as np
import pytest
import torch

from oracle import hg_oracle as O
from oracle import hg_policy as P
from paper_2604_18529_b200 import hybrid
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import LSE_ABS, OUT_MAX_ABS, OUT_REL_L2, bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def reference(w, q, K, V, idx, n_sel, G):
    out = np.zeros((w.B, w.Hq, w.D)); lse = np.zeros((w.B, w.Hq))
    for b in range(w.B):
        for h in range(w.Hq):
            g = h // G
            host = idx[b, g, : int(n_sel[b])].numpy().astype(np.int64)
            assert len(set(host.tolist())) == len(host) and (host >= 0).all() and (host < w.tok_begin[b]).all()
            tokens = np.concatenate([host, np.arange(w.tok_begin[b], w.tok_end[b])])
            out[b, h], lse[b, h] = O.full(q[b, h], np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g]),
                                          w.dtype, idx=tokens)
    return out, lse


@pytest.mark.parametrize("G,dtype", [(1, "f16"), (4, "bf16")])
def test_hybrid_steps_match_attention_over_the_tokens_they_used(G, dtype):
    w = W.AttnWorkload("hyb", 2, 2 * G, 2, 128, dtype, [1500, 700], [1100, 420], [1500, 700], page_size=16,
                       chunk_tokens=128, seed=90 + G, outlier_frac=0.02)
    q_t, K_t, V_t = w.q(), w.kv_logical("k"), w.kv_logical("v")
    prob = DeviceProblem(w, DEV)
    n_host = torch.tensor(w.tok_begin, dtype=torch.int32)                 # the host holds [0, tok_begin)
    eng = hybrid.HybridAttentionStep(prob.desc, K_t, V_t, n_host, k_min=32, k_max=160, k_step=32, sinks=4,
                                     handoff_chunk=64, host_threads=2, device=DEV)
    q, K, V = bits(q_t), bits(K_t), bits(V_t)
    seen = set()
    for step in range(8):
        if step == 4:                                                     # force the other strategy for the rest
            eng.set_operating_point(eng.k, hybrid.PRE_QK if eng.strategy == hybrid.POST_QK else hybrid.POST_QK)
        k_used, strat_used = eng.k, eng.strategy
        with torch.cuda.device(DEV):
            rec = eng.step(prob.q, q_t, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                           prob.out, prob.lse)
        assert (rec.k, rec.strategy) == (k_used, strat_used)
        assert rec.t_gpu > 0 and rec.t_cpu > 0 and rec.t_tx > 0 and rec.t_step >= rec.t_cpu
        assert eng.idx.shape == (w.B, w.Hkv, k_used)
        assert [int(x) for x in eng.n_sel] == [min(k_used, n) for n in w.tok_begin]
        if strat_used == hybrid.PRE_QK:                                   # sinks + the most recent host tokens
            for b in range(w.B):
                want = P.positions(w.tok_begin[b], 4, max(k_used - 4, 0), k_used)
                assert eng.idx[b, 0, : len(want)].tolist() == want
        ref_out, ref_lse = reference(w, q, K, V, eng.idx, eng.n_sel, G)
        out, lse = prob.out.double().cpu().numpy(), prob.lse.double().cpu().numpy()
        assert np.abs(out - ref_out).max() <= OUT_MAX_ABS
        assert np.linalg.norm(out - ref_out) / np.linalg.norm(ref_out) <= OUT_REL_L2
        assert np.abs(lse - ref_lse).max() <= LSE_ABS
        # Algorithm 1 on the latencies this step measured gives the next step's K and strategy
        assert (eng.k, eng.strategy) == P.feedback_scheduler_step(k_used, strat_used, rec.t_gpu, rec.t_cpu, rec.t_tx, 32, 160, 32)
        seen.add(strat_used)
    assert seen == {hybrid.POST_QK, hybrid.PRE_QK}
    assert len(eng.history) == 8


def test_post_qk_picks_the_heaviest_host_tokens():
    """With a few host tokens made to dominate (keys aligned with the query), Post-QK^T selection finds them."""
    w = W.AttnWorkload("heavy", 1, 2, 2, 128, "f16", [900], [600], [900], page_size=16, chunk_tokens=128, seed=5)
    q_t, K_t, V_t = w.q(), w.kv_logical("k").clone(), w.kv_logical("v")
    heavy = [17, 250, 333, 599]
    for g in range(w.Hkv):
        for t in heavy:
            K_t[0, t, g] = (q_t[0, g].float() * 3).half()                   # logit = 3 |q|^2 / sqrt(D): far above the rest
    prob = DeviceProblem(w, DEV)
    eng = hybrid.HybridAttentionStep(prob.desc, K_t, V_t, torch.tensor([600], dtype=torch.int32), k_min=8, k_max=8, k_step=8,
                                     handoff_chunk=32, device=DEV)
    with torch.cuda.device(DEV):
        eng.step(prob.q, q_t, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, prob.out, prob.lse)
    for g in range(w.Hkv):
        assert set(heavy) <= set(eng.idx[0, g].tolist())


def test_decode_loop_with_append_eviction_and_exact_hybrid_attention():
    """The cache's whole life: every step appends the new token's K/V on the GPU; when a slice outgrows its
    budget the oldest tokens move to the host store; attention is the hybrid step with K large enough to take
    every host token, so each step must equal monolithic attention over the whole sequence so far."""
    import paper_2604_18529_b200 as pkg
    from test_kv_residency_gpu import poison_future_rows, rows_at
    G, steps, budget, evict_n = 2, 12, 200, 64
    final = W.AttnWorkload("loop", 2, 2 * G, 2, 128, "f16", [400, 260], [0, 0], [400, 260], page_size=16, chunk_tokens=128,
                           seed=123)
    start = [L - steps for L in final.seq_lens]
    prob = DeviceProblem(final, DEV)                      # pool and block table sized for the final lengths
    poison_future_rows(prob, final, start)
    prob.seq_lens = torch.tensor(start, dtype=torch.int32, device=DEV)
    prob.tok_end = torch.tensor(start, dtype=torch.int32, device=DEV)
    store = hybrid.HostKvStore(final.B, 512, final.Hkv, final.D, torch.float16)
    eng = hybrid.HybridAttentionStep(prob.desc, store.k, store.v, store.n, k_min=512, k_max=512, k_step=64, handoff_chunk=128,
                                     device=DEV)
    q_t = final.q()
    q, K, V = bits(q_t), bits(final.kv_logical("k")), bits(final.kv_logical("v"))
    tb = [0, 0]
    evictions = 0
    with torch.cuda.device(DEV):
        for s in range(steps):
            t_new = [a + s for a in start]
            pkg.hg_kv_append(rows_at(final, "k", t_new), rows_at(final, "v", t_new), prob.kv["k"], prob.kv["v"],
                             prob.seq_lens, prob.tok_end, prob.desc)
            lens = [t + 1 for t in t_new]
            n_evict = [evict_n if lens[b] - tb[b] > budget else 0 for b in range(final.B)]
            if any(n_evict):
                store.evict_from_gpu(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, n_evict, prob.desc)
                tb = [a + n for a, n in zip(tb, n_evict)]
                eng.set_host_tokens(store.n)
                evictions += 1
            assert prob.tok_begin.tolist() == tb == store.n.tolist() and prob.tok_end.tolist() == lens
            for b in range(final.B):                      # the host rows are the sequence's prefix, bit for bit
                for g in range(final.Hkv):
                    assert torch.equal(store.k[b, : tb[b], g], final.kv_rows("k", b, g, 0, tb[b]))
                    assert torch.equal(store.v[b, : tb[b], g], final.kv_rows("v", b, g, 0, tb[b]))
            eng.set_operating_point(512, hybrid.POST_QK if s % 2 == 0 else hybrid.PRE_QK)
            eng.step(prob.q, q_t, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, prob.out, prob.lse)
            assert int(prob.status.item()) == 0
            ref_out, ref_lse = O.full_batch(q, K, V, final.dtype, [0, 0], lens)
            out, lse = prob.out.double().cpu().numpy(), prob.lse.double().cpu().numpy()
            assert np.abs(out - ref_out).max() <= OUT_MAX_ABS, s
            assert np.linalg.norm(out - ref_out) / np.linalg.norm(ref_out) <= OUT_REL_L2, s
            assert np.abs(lse - ref_lse).max() <= LSE_ABS, s
    assert evictions >= 3 and tb[0] > tb[1] >= 0


def test_pre_qk_selection_from_a_callers_ranking():
    """The token selector takes any ranked candidate list (Section 4.5): here a list built from an earlier
    Post-QK^T step's choice, padded with -1 where a head has fewer candidates."""
    G = 2
    w = W.AttnWorkload("rank", 2, 2 * G, 2, 128, "f16", [1200, 500], [800, 300], [1200, 500], page_size=16,
                       chunk_tokens=128, seed=77)
    q_t, K_t, V_t = w.q(), w.kv_logical("k"), w.kv_logical("v")
    prob = DeviceProblem(w, DEV)
    eng = hybrid.HybridAttentionStep(prob.desc, K_t, V_t, torch.tensor(w.tok_begin, dtype=torch.int32), k_min=48, k_max=48,
                                     k_step=16, handoff_chunk=32, device=DEV)
    q, K, V = bits(q_t), bits(K_t), bits(V_t)
    args = (prob.q, q_t, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, prob.out, prob.lse)
    with torch.cuda.device(DEV):
        eng.step(*args)                                            # Post-QK^T: the 48 best per KV head
        ranking = torch.full((w.B, w.Hkv, 64), -1, dtype=torch.int32)
        ranking[:, :, :48] = eng.idx.flip(2)                       # some order; what matters is which 48 come first
        ranking[1, 1, 40:] = -1                                    # one head of sequence 1 offers only 40
        eng.set_pre_qk_ranking(ranking)
        eng.set_operating_point(48, hybrid.PRE_QK)
        eng.step(*args)
    assert eng.n_sel.tolist() == [48, 40]
    assert torch.equal(eng.idx[0], ranking[0, :, :48]) and torch.equal(eng.idx[1, :, :40], ranking[1, :, :40])
    ref_out, ref_lse = reference(w, q, K, V, eng.idx, eng.n_sel, G)
    out, lse = prob.out.double().cpu().numpy(), prob.lse.double().cpu().numpy()
    assert np.abs(out - ref_out).max() <= OUT_MAX_ABS and np.abs(lse - ref_lse).max() <= LSE_ABS
    with torch.cuda.device(DEV):
        eng.set_pre_qk_ranking(None)                               # back to sinks + recent window
        eng.set_operating_point(48, hybrid.PRE_QK)
        eng.step(*args)
    assert eng.idx[0, 0, :4].tolist() == [0, 1, 2, 3] and eng.n_sel.tolist() == [48, 48]


def test_host_store_on_bound_and_registered_tier_memory():
    """K rows and V rows of the host tier bound to NUMA nodes (node 0 for both here: one node is all this machine
    has) and registered with the CUDA runtime: eviction lands in them and the hybrid step reads them."""
    import paper_2604_18529_b200 as pkg
    G = 2
    w = W.AttnWorkload("tier", 2, 2 * G, 2, 128, "f16", [500, 260], [0, 0], [500, 260], page_size=16, chunk_tokens=128, seed=321)
    prob = DeviceProblem(w, DEV)
    store = hybrid.HostKvStore(w.B, 256, w.Hkv, w.D, torch.float16, k_node=0, v_node=0)
    with torch.cuda.device(DEV):
        store.evict_from_gpu(prob.kv["k"], prob.kv["v"], prob.tok_begin, prob.tok_end, [200, 100], prob.desc)
        assert prob.tok_begin.tolist() == [200, 100] == store.n.tolist()
        for b in range(w.B):
            for g in range(w.Hkv):
                assert torch.equal(store.k[b, : int(store.n[b]), g], w.kv_rows("k", b, g, 0, int(store.n[b])))
        assert store._tiers[0].node_of() == 0 and store._tiers[1].node_of() == 0
        eng = hybrid.HybridAttentionStep(prob.desc, store.k, store.v, store.n, k_min=256, k_max=256, k_step=64, handoff_chunk=128,
                                         device=DEV)
        eng.step(prob.q, w.q(), prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, prob.out, prob.lse)
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    ref_out, ref_lse = O.full_batch(q, K, V, w.dtype, [0, 0], w.seq_lens)
    out, lse = prob.out.double().cpu().numpy(), prob.lse.double().cpu().numpy()
    assert np.abs(out - ref_out).max() <= OUT_MAX_ABS and np.abs(lse - ref_lse).max() <= LSE_ABS
    del eng
    for t in store._tiers:
        t.free()


def test_layer_pipeline_overlaps_cpu_stages_and_gives_the_same_results():
    """Three layers (same cache, a query per layer): with the CPU stage of layer i + 1 running on a host thread
    while the GPU handles layer i, every layer's result is what the layer-after-layer order gives, and equals
    attention over the GPU slice plus the tokens that layer chose; one (K, strategy) per pass."""
    G, L = 2, 3
    w = W.AttnWorkload("pipe", 2, 2 * G, 2, 128, "f16", [1300, 600], [900, 350], [1300, 600], page_size=16,
                       chunk_tokens=128, seed=555)
    K_t, V_t = w.kv_logical("k"), w.kv_logical("v")
    prob = DeviceProblem(w, DEV)
    n_host = torch.tensor(w.tok_begin, dtype=torch.int32)
    gen = torch.Generator().manual_seed(3)
    q_host = [torch.randn(w.B, w.Hq, w.D, generator=gen).half() for _ in range(L)]
    q_dev = [q.to(DEV) for q in q_host]
    kv = [(prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end)] * L
    layers = [hybrid.HybridAttentionStep(prob.desc, K_t, V_t, n_host, k_min=64, k_max=128, k_step=32, handoff_chunk=64,
                                         host_threads=2, device=DEV) for _ in range(L)]
    pipe = hybrid.HybridPipeline(layers)
    Kb, Vb = bits(K_t), bits(V_t)
    results = {}
    for pipelined in (False, True):
        for e in layers:
            e.set_operating_point(64, hybrid.POST_QK)
        outs = [(torch.empty_like(prob.out), torch.empty_like(prob.lse)) for _ in range(L)]
        with torch.cuda.device(DEV):
            ms = pipe.run(q_dev, q_host, kv, outs, pipelined=pipelined)
        assert ms > 0
        recs = [e.history[-1] for e in layers]
        assert all(r.k == 64 and r.strategy == hybrid.POST_QK for r in recs)
        mean = lambda f: sum(getattr(r, f) for r in recs) / L
        want = P.feedback_scheduler_step(64, hybrid.POST_QK, mean("t_gpu"), mean("t_cpu"), mean("t_tx"), 64, 128, 32)
        assert all((e.k, e.strategy) == want for e in layers)              # one operating point for all layers
        for i, e in enumerate(layers):
            ref_out, ref_lse = reference(w, bits(q_host[i]), Kb, Vb, e.idx, e.n_sel, G)
            out, lse = outs[i][0].double().cpu().numpy(), outs[i][1].double().cpu().numpy()
            assert np.abs(out - ref_out).max() <= OUT_MAX_ABS and np.abs(lse - ref_lse).max() <= LSE_ABS
        results[pipelined] = [(o.clone(), l.clone()) for o, l in outs]
    for (o0, l0), (o1, l1) in zip(results[False], results[True]):
        assert torch.equal(o0, o1) and torch.equal(l0, l1)

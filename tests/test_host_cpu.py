"""Host-side companions (logits calculator, selection, gather, feedback scheduler) against the oracle and the
plain statements in oracle/hg_policy.py.  CPU only."""
import itertools

import numpy as np
import pytest
import torch

from oracle import hg_oracle as O
from oracle import hg_policy as P
from paper_2604_18529_b200 import build as hgbuild
from paper_2604_18529_b200 import host as H
from paper_2604_18529_b200 import workload as W


@pytest.fixture(scope="module", autouse=True)
def _built():
    hgbuild.build()


def bits(t):
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


@pytest.mark.parametrize("dtype,D,G", [("f16", 128, 1), ("bf16", 64, 4), ("f16", 64, 3), ("f16", 128, 8), ("bf16", 40, 2),
                                       ("f16", 320, 1)])
def test_host_logits_match_the_oracle(dtype, D, G):
    w = W.AttnWorkload("h", 2, 2 * G, 2, D, dtype, [300, 170], [200, 170], [300, 170], seed=3, sigma_kv=1.5)
    q, K = w.q(), w.kv_logical("k")                         # [B][Hq][D], [B][Lmax][Hkv][D]
    n_host = torch.tensor(w.tok_begin, dtype=torch.int32)   # the host holds [0, tok_begin)
    Ksel = int(n_host.max())
    desc = H.host_desc(K, w.Hq, Ksel, threads=3)
    logits = torch.empty(w.B, w.Hq, Ksel)
    H.hg_host_logits(q, K, None, n_host, logits, desc)
    qb, Kb = bits(q), bits(K)
    for b in range(w.B):
        for h in range(w.Hq):
            want = O.logits(qb[b, h], np.ascontiguousarray(Kb[b, :, h // G]), dtype, t0=0, n=int(n_host[b]))
            got = logits[b, h, : int(n_host[b])].double().numpy()
            assert np.abs(got - want).max() <= 2e-5 * max(1.0, np.abs(want).max())
            assert torch.isinf(logits[b, h, int(n_host[b]):]).all()
    # through an index list, with an explicit scale
    idx = torch.stack([torch.stack([torch.randperm(Ksel, generator=torch.Generator().manual_seed(b * 7 + g))[:50]
                                    for g in range(w.Hkv)]) for b in range(w.B)]).to(torch.int32)
    idx[1] = idx[1] % max(int(n_host[1]), 1)
    n_sel = torch.tensor([50, 37], dtype=torch.int32)
    desc2 = H.host_desc(K, w.Hq, 50, scale=0.25)
    lg2 = torch.empty(w.B, w.Hq, 50)
    H.hg_host_logits(q, K, idx, n_sel, lg2, desc2)
    for b in range(w.B):
        for h in range(w.Hq):
            n = int(n_sel[b])
            want = O.logits(qb[b, h], np.ascontiguousarray(Kb[b, :, h // G]), dtype, scale=0.25, idx=idx[b, h // G, :n].numpy())
            assert np.abs(lg2[b, h, :n].double().numpy() - want).max() <= 2e-5 * max(1.0, np.abs(want).max())


def test_host_logits_head_major_rows_give_the_same_bits():
    """Rows stored [B][Hkv][T][D] (each KV head a stream of its own) take the other split of the work; the
    arithmetic per (token, head) is the same, so the logits are bit-identical to the token-major call."""
    w = W.AttnWorkload("h", 2, 8, 2, 128, "f16", [700, 333], [650, 301], [700, 333], seed=8)
    q, K = w.q(), w.kv_logical("k")
    n_host = torch.tensor(w.tok_begin, dtype=torch.int32)
    Ksel = int(n_host.max())
    a = torch.empty(w.B, w.Hq, Ksel)
    H.hg_host_logits(q, K, None, n_host, a, H.host_desc(K, w.Hq, Ksel, threads=2))
    K_hm = K.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)        # same shape, head-major storage
    assert K_hm.stride(2) > K_hm.stride(1)
    b = torch.empty(w.B, w.Hq, Ksel)
    H.hg_host_logits(q, K_hm, None, n_host, b, H.host_desc(K_hm, w.Hq, Ksel, threads=5))
    assert torch.equal(a, b)


def test_host_logits_from_two_caller_threads_at_once():
    """The worker pool serves one call at a time; a call that finds it busy runs on threads of its own.
    Either way the result is the same."""
    import threading
    w = W.AttnWorkload("h", 4, 8, 4, 128, "bf16", [3000] * 4, [2900] * 4, [3000] * 4, seed=12)
    q, K = w.q(), w.kv_logical("k")
    n_host = torch.tensor(w.tok_begin, dtype=torch.int32)
    want = torch.empty(w.B, w.Hq, 2900)
    H.hg_host_logits(q, K, None, n_host, want, H.host_desc(K, w.Hq, 2900, threads=1))
    outs = [torch.empty(w.B, w.Hq, 2900) for _ in range(4)]

    def call(o):
        for _ in range(5):
            H.hg_host_logits(q, K, None, n_host, o, H.host_desc(K, w.Hq, 2900, threads=4))

    ts = [threading.Thread(target=call, args=(o,)) for o in outs]
    for t in ts:
        t.start()
    for t in ts:
        t.join()
    for o in outs:
        assert torch.equal(o, want)


def test_topk_selection_matches_the_sort_definition():
    rng = np.random.default_rng(5)
    scores = rng.standard_normal((6, 200)).astype(np.float32)
    scores[0, 10:20] = scores[0, 5]                       # ties
    scores[1, 3] = np.nan
    scores[2, :] = -np.inf
    n = np.array([200, 200, 200, 0, 7, 150], dtype=np.int32)
    for k in (1, 5, 64, 300):
        idx, n_out = H.hg_host_select_topk(torch.from_numpy(scores), torch.from_numpy(n), k)
        for r in range(6):
            want = P.topk(list(scores[r, : n[r]]), k)
            assert int(n_out[r]) == len(want)
            assert idx[r, : len(want)].tolist() == want and (idx[r, len(want):] == -1).all()


def test_topk_with_many_ties_and_nans_matches_the_sort_definition():
    rng = np.random.default_rng(1)
    for trial in range(30):
        rows, stride = 5, int(rng.integers(1, 300))
        sc = rng.integers(-3, 4, (rows, stride)).astype(np.float32)          # seven distinct values: ties everywhere
        sc[rng.random((rows, stride)) < 0.05] = np.nan
        n = rng.integers(0, stride + 1, rows).astype(np.int32)
        k = int(rng.integers(1, 40))
        idx, n_out = H.hg_host_select_topk(torch.from_numpy(sc), torch.from_numpy(n), k)
        for r in range(rows):
            want = P.topk(list(sc[r, : n[r]]), k)
            assert [i for i in idx[r].tolist() if i >= 0] == want and int(n_out[r]) == len(want)
            assert idx[r, len(want):].tolist() == [-1] * (k - len(want))


def test_group_scores_and_logit_gather():
    rng = np.random.default_rng(9)
    rows, group, stride = 6, 3, 41
    lg = rng.standard_normal((rows * group, stride)).astype(np.float32)
    lg[4, 7] = np.nan                                         # a NaN loses to any number
    n = np.array([41, 0, 17, 41, 1, 30], dtype=np.int32)
    got = H.hg_host_group_scores(torch.from_numpy(lg), group, torch.from_numpy(n)).numpy()
    for r in range(rows):
        want = np.fmax.reduce(lg[r * group:(r + 1) * group, : n[r]], axis=0) if n[r] else np.empty(0)
        assert np.array_equal(got[r, : n[r]], want)
        assert np.isneginf(got[r, n[r]:]).all()
    # gather: [B][Hq][full] -> [B][Hq][K] through idx [B][Hkv][K]
    B, Hkv, G, D, full, K = 2, 2, 3, 64, 50, 8
    fl = torch.from_numpy(rng.standard_normal((B, Hkv * G, full)).astype(np.float32))
    idx = torch.from_numpy(rng.integers(0, full, (B, Hkv, K)).astype(np.int32))
    idx[1, 0, 2] = full + 3                                   # out of range: -inf, never read
    n_sel = torch.tensor([8, 5], dtype=torch.int32)
    desc = H.host_desc(torch.zeros(B, 1, Hkv, D, dtype=torch.float16), Hkv * G, K)
    out = torch.empty(B, Hkv * G, K)
    H.hg_host_gather_logits(fl, idx, n_sel, out, desc)
    for b in range(B):
        for h in range(Hkv * G):
            for i in range(K):
                j = int(idx[b, h // G, i])
                want = fl[b, h, j].item() if i < int(n_sel[b]) and 0 <= j < full else -np.inf
                assert out[b, h, i].item() == want


def test_position_selection():
    for n_tokens, sinks, window, k in itertools.product([0, 1, 5, 100, 2000], [0, 4], [0, 3, 1024], [1, 6, 5000]):
        got = H.hg_host_select_positions(n_tokens, sinks, window, k).tolist()
        assert got == P.positions(n_tokens, sinks, window, k) if n_tokens > 0 else got == []
    assert H.hg_host_select_positions(2000, 4, 1024, 1028).tolist() == list(range(4)) + list(range(976, 2000))


def test_gather_rows():
    w = W.AttnWorkload("g", 2, 4, 2, 64, "bf16", [90, 60], [0, 0], [90, 60], seed=9)
    V = w.kv_logical("v")
    K = 11
    idx = torch.tensor([[[5, 0, 89, 3, 3, 7, 1, 2, 4, 6, 8], [1] * 11], [[59, 58, 0, 1, 2, 3, 4, 5, 6, 7, 8], [9] * 11]], dtype=torch.int32)
    n_sel = torch.tensor([11, 4], dtype=torch.int32)
    dst = torch.full((2, 2, K, 64), 1.0, dtype=torch.bfloat16)
    H.hg_host_gather_rows(V, idx, n_sel, dst, H.host_desc(V, 4, K))
    for b in range(2):
        for g in range(2):
            n = int(n_sel[b])
            assert torch.equal(dst[b, g, :n], V[b, idx[b, g, :n].long(), g])
            assert (dst[b, g, n:] == 0).all()


def test_gather_rows_never_reads_outside_the_buffer():
    """Selections are -1 padded, and a caller may pass a count that reaches into the padding: such slots (and
    indices at or beyond the stated number of rows) come back as zero rows instead of an out-of-bounds read."""
    w = W.AttnWorkload("g2", 1, 2, 1, 64, "f16", [40], [0], [40], seed=10)
    V = w.kv_logical("v")
    idx = torch.tensor([[[3, -1, 39, 40, 7, 1 << 20]]], dtype=torch.int32)
    dst = torch.full((1, 1, 6, 64), 1.0, dtype=torch.float16)
    H.hg_host_gather_rows(V, idx, torch.tensor([6], dtype=torch.int32), dst, H.host_desc(V, 2, 6))
    assert torch.equal(dst[0, 0, 0], V[0, 3, 0]) and torch.equal(dst[0, 0, 2], V[0, 39, 0]) and torch.equal(dst[0, 0, 4], V[0, 7, 0])
    assert (dst[0, 0, [1, 3, 5]] == 0).all()


def test_feedback_scheduler_follows_algorithm_1():
    rng = np.random.default_rng(11)
    k_min, k_max, step = 128, 1024, 96
    s = H.FeedbackScheduler(k_min, k_max, step)
    k, strat = P.feedback_scheduler_init(k_min)
    assert (s.state.k, s.state.strategy) == (k, strat) == (128, P.POST_QK)
    for _ in range(400):
        t_gpu, t_cpu, t_tx = rng.uniform(0.5, 2.0), rng.uniform(0.1, 2.0), rng.uniform(0.0, 0.5)
        k, strat = P.feedback_scheduler_step(k, strat, t_gpu, t_cpu, t_tx, k_min, k_max, step)
        assert s.update(t_gpu, t_cpu, t_tx) == (k, strat)
        assert k_min <= k <= k_max
    # the listing's cases, one by one
    s = H.FeedbackScheduler(128, 1024, 100)
    assert s.update(1.0, 0.5, 0.2) == (228, H.HG_SCHED_POST_QK)          # hidden: K grows
    assert s.update(1.0, 0.9, 0.2) == (128, H.HG_SCHED_POST_QK)          # not hidden, K > K_min: shrink, clamped
    assert s.update(1.0, 0.9, 0.2) == (128, H.HG_SCHED_PRE_QK)           # at K_min: switch strategy
    assert s.update(1.0, 0.5, 0.5) == (228, H.HG_SCHED_PRE_QK)           # boundary t_cpu + t_tx == t_gpu counts as hidden:
    for _ in range(20):                                                  # K grows, the strategy is not set back
        s.update(1.0, 0.1, 0.1)
    assert (s.state.k, s.state.strategy) == (1024, H.HG_SCHED_PRE_QK)


def test_tier_memory_is_bound_to_its_node():
    assert H.hg_host_tier_nodes() >= 1
    buf = H.TierBuffer((3, 1000, 64), torch.float16, node=0)
    assert buf.node_of() == -1                                  # nothing touched yet: no page behind it
    buf.tensor.fill_(1.5)
    assert buf.node_of() == 0 and buf.node_of(buf.nbytes - 1) == 0
    assert buf.tensor.shape == (3, 1000, 64) and float(buf.tensor.float().sum()) == 1.5 * 3 * 1000 * 64
    buf.free()
    with pytest.raises(H.HgError):
        H.TierBuffer((16,), torch.float32, node=H.hg_host_tier_nodes() + 500)   # no such node
    with pytest.raises(H.HgError):
        H.TierBuffer((16,), torch.float32, node=-1)


def test_ranked_selection_against_the_policy_oracle():
    rng = np.random.default_rng(21)
    for _ in range(60):
        B, Hkv, R = int(rng.integers(1, 4)), int(rng.integers(1, 4)), int(rng.integers(1, 12))
        n_host = [int(rng.integers(0, 15)) for _ in range(B)]
        k = int(rng.integers(1, 14))
        ranking = torch.full((B, Hkv, R), -1, dtype=torch.int32)
        for b in range(B):
            for g in range(Hkv):
                n = int(rng.integers(0, R + 1))
                ranking[b, g, :n] = torch.from_numpy(rng.integers(0, 16, size=n).astype(np.int32))   # now and then >= n_host
        idx, n = H.hg_host_select_ranked(ranking, torch.tensor(n_host, dtype=torch.int32), k)
        for b in range(B):
            want = P.ranked([ranking[b, g].tolist() for g in range(Hkv)], k, n_host[b])
            assert int(n[b]) == len(want[0])
            for g in range(Hkv):
                assert idx[b, g].tolist() == want[g] + [-1] * (k - len(want[g]))

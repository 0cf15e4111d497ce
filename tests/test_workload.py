"""The seeded input generator: determinism, value distribution, and that the paged pools, the block
table and the logical rows describe the same cache.  CPU only."""
import dataclasses

import pytest
import torch

from paper_2604_18529_b200 import workload as W


def small(**kw):
    base = dict(name="t", B=2, Hq=4, Hkv=2, D=64, dtype="f16", seq_lens=[150, 97], tok_begin=[37, 0],
                tok_end=[150, 60], page_size=16, layout="HND", chunk_tokens=64, seed=7)
    base.update(kw)
    return W.AttnWorkload(**base)


def test_hash_matches_python_integers():
    key = W.tensor_key(5, W.TENSOR_K)
    idx = torch.tensor([0, 1, 2, 12345678901, (1 << 40) + 17], dtype=torch.int64)
    got = W.hash64(key, idx).tolist()
    for i, g in zip(idx.tolist(), got):
        assert (g & ((1 << 64) - 1)) == W._mix_int(key + i * W._GOLDEN)


def test_values_are_standard_normal_and_seeded():
    w = small(B=1, Hq=2, Hkv=2, seq_lens=[4096], tok_begin=[0], tok_end=[4096])
    k = w.kv_rows("k", 0, 1, 0, 4096).float()
    assert abs(k.mean().item()) < 0.01 and abs(k.std().item() - 1.0) < 0.01
    assert torch.equal(w.kv_rows("k", 0, 1, 100, 200), w.kv_rows("k", 0, 1, 0, 4096)[100:200])
    assert not torch.equal(w.kv_rows("k", 0, 1, 0, 64), w.kv_rows("v", 0, 1, 0, 64))
    assert not torch.equal(w.kv_rows("k", 0, 0, 0, 64), w.kv_rows("k", 0, 1, 0, 64))
    w2 = dataclasses.replace(w, seed=8)
    assert not torch.equal(w.kv_rows("k", 0, 0, 0, 64), w2.kv_rows("k", 0, 0, 0, 64))
    half = dataclasses.replace(w, sigma_kv=0.5)
    assert abs(half.kv_rows("v", 0, 0, 0, 4096).float().std().item() - 0.5) < 0.01


def test_outlier_tokens_scale_k_and_v_rows_for_every_head():
    w = small(B=1, Hq=2, Hkv=2, seq_lens=[20000], tok_begin=[0], tok_end=[20000], outlier_frac=0.01)
    plain = dataclasses.replace(w, outlier_frac=0.0)
    k0, k1 = plain.kv_rows("k", 0, 0, 0, 20000).float(), w.kv_rows("k", 0, 0, 0, 20000).float()
    ratio = (k1.abs().sum(1) / k0.abs().sum(1))
    is_out = ratio > 4
    assert 0.006 < is_out.float().mean().item() < 0.014
    assert torch.allclose(ratio[~is_out], torch.ones_like(ratio[~is_out]))
    for which, g in (("v", 0), ("k", 1), ("v", 1)):
        a, b = plain.kv_rows(which, 0, g, 0, 20000).float(), w.kv_rows(which, 0, g, 0, 20000).float()
        assert torch.equal((b.abs().sum(1) / a.abs().sum(1)) > 4, is_out)


@pytest.mark.parametrize("layout,paged", [("HND", True), ("NHD", True), ("NHD", False)])
def test_device_pools_hold_the_logical_rows(layout, paged):
    w = small(layout=layout, paged=paged)
    kv = w.build_device_kv("cpu")
    ps = w.page_size
    for which in ("k", "v"):
        pool = kv[which].reshape(-1)
        for b in range(w.B):
            for g in range(w.Hkv):
                rows = w.kv_rows(which, b, g, 0, w.seq_lens[b])
                for t in range(w.tok_begin[b], w.tok_end[b]):
                    page = t // ps
                    phys = kv["block_table"][b, page].item() if paged else b * kv["max_pages"] + page
                    assert phys >= 0
                    off = phys * kv["page_stride"] + g * kv["head_stride"] + (t % ps) * kv["tok_stride"]
                    assert torch.equal(pool[off:off + w.D], rows[t])
    if paged:
        table = kv["block_table"]
        assert kv["num_pages"] == (table >= 0).sum().item()
        assert sorted(table[table >= 0].tolist()) == list(range(kv["num_pages"]))
        # pages that hold no GPU token are not resident
        assert table[0, 0].item() == -1 and table[0, 37 // ps].item() >= 0


def test_chunk_grid_is_absolute_and_clipped():
    w = small()
    assert w.chunk_grid(0) == (0, 3)            # [37,150) over 64-token chunks: 0..2
    assert [w.chunk_range(0, c) for c in range(4)] == [(37, 64), (64, 128), (128, 150), (0, 0)]
    assert w.chunk_grid(1) == (0, 1) and w.chunk_range(1, 0) == (0, 60)
    assert w.num_chunks == 3
    e = small(tok_begin=[150, 10], tok_end=[150, 10])
    assert e.num_chunks == 1 and e.chunk_grid(0) == (0, 0) and e.gpu_tokens == 0


def test_benchmark_configurations_have_the_stated_shapes():
    t = W.make_workload("tiny")
    assert (t.B, t.Hq, t.Hkv, t.D, t.seq_lens, t.tok_begin, t.tok_end) == (1, 8, 8, 64, [2048], [0], [1024])
    o = W.make_workload("opt13b")
    assert o.gpu_tokens == 8 * 19660 and o.tok_begin[0] == 13108 and o.kv_bytes() == 3221094400
    p = W.make_workload("opt30b")
    assert p.dtype == "bf16" and p.gpu_tokens == 4 * 65536 and p.page_size == 64 and p.chunk_tokens == 2048
    l = W.make_workload("llama70b")
    assert (l.Hq, l.Hkv, l.gpu_tokens) == (64, 8, 419430)
    r = W.make_workload("ragged")
    assert r.B == 16 and all(4096 <= x <= 65536 for x in r.seq_lens)
    assert all(0.1 <= (e - b) / L <= 0.9 + 1e-9 for b, e, L in zip(r.tok_begin, r.tok_end, r.seq_lens))
    assert r.tok_end == r.seq_lens
    for name in W.WORKLOADS:
        s = W.scaled_down(W.make_workload(name), 64)
        assert s.G == W.make_workload(name).G and s.gpu_tokens > 0

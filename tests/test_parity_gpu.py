"""GPU path vs the fp64 oracle, element by element, through the C ABI (via the thin binding).

Sizes are small enough for the whole-tensor oracle yet span several 64-token tiles, several chunks
and ragged first/last tiles.  Tolerances (parity_util): out max-abs 2e-3, rel-L2 1e-3, LSE 1e-4.
"""
import dataclasses

import numpy as np
import pytest
import torch

import paper_2604_18529_b200 as pkg
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import OracleRef, bits, check_output, check_partials

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_and_check(w, poison_tail=False, what=None, **tune):
    what = what or w.name
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV, poison_tail=poison_tail)
    if tune:
        prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, **tune)
    prob.partial()
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK, what
    rm, rl, ro = ref.chunk_partials(w.chunk_tokens, prob.NC)
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D), what)
    prob.merge(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    return prob, ref, check_output(prob.out, prob.lse, ref.out, ref.lse, what)


def wl(**kw):
    base = dict(name="case", B=2, Hq=4, Hkv=2, D=128, dtype="f16", seq_lens=[700, 333], tok_begin=[130, 5],
                tok_end=[700, 290], page_size=16, layout="HND", chunk_tokens=128, seed=11)
    base.update(kw)
    return W.AttnWorkload(**base)


# ---- the five benchmark configurations, scaled down ------------------------------------------------

@pytest.mark.parametrize("name", W.WORKLOADS)
def test_scaled_down_benchmark_configs(name):
    full = W.make_workload(name)
    w = full if name == "tiny" else W.scaled_down(full, 64 if name != "ragged" else 16, max_batch=3)
    run_and_check(w)


# ---- shape sweep: head grouping, head_dim, dtype, page size, layout ----------------------------------

@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (3, 3), (4, 1), (8, 1), (6, 2), (16, 1), (12, 1)])
@pytest.mark.parametrize("D", [64, 128])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_head_grouping_sweep(Hq, Hkv, D, dtype):
    run_and_check(wl(Hq=Hq, Hkv=Hkv, D=D, dtype=dtype, seed=100 + Hq * 7 + D))


@pytest.mark.parametrize("page_size", [16, 32, 64, 128, 256])
@pytest.mark.parametrize("layout,paged", [("HND", True), ("NHD", True), ("NHD", False)])
@pytest.mark.parametrize("G", [1, 4])
def test_page_size_and_layout_sweep(page_size, layout, paged, G):
    chunk = max(128, page_size)
    w = wl(Hq=2 * G, Hkv=2, page_size=page_size, layout=layout, paged=paged, chunk_tokens=chunk,
           seq_lens=[900, 517], tok_begin=[77, 0], tok_end=[900, 400], seed=page_size + G)
    run_and_check(w)


@pytest.mark.parametrize("G", [1, 8])
@pytest.mark.parametrize("chunk", [64, 192, 256, 1024])
def test_chunk_sizes(G, chunk):
    w = wl(Hq=G, Hkv=1, chunk_tokens=chunk, seq_lens=[1500, 64], tok_begin=[333, 0], tok_end=[1500, 64], seed=chunk)
    run_and_check(w)


# ---- edge cases ---------------------------------------------------------------------------------------

@pytest.mark.parametrize("G", [1, 4])
@pytest.mark.parametrize("tb,te,L", [
    (0, 0, 100),          # empty slice at the start
    (100, 100, 100),      # empty slice at the end
    (37, 38, 100),        # one token
    (64, 128, 300),       # exactly one aligned tile
    (63, 65, 300),        # two tokens straddling a tile boundary
    (0, 300, 300),        # everything on the GPU, nothing on the host
    (17, 29, 300),        # inside one page
    (127, 129, 130),      # straddles a chunk boundary
])
def test_slice_edge_cases(G, tb, te, L):
    w = wl(B=2, Hq=2 * G, Hkv=2, seq_lens=[L, 200], tok_begin=[tb, 10], tok_end=[te, 150], chunk_tokens=128, seed=tb + te)
    run_and_check(w, what=f"G{G} [{tb},{te}) of {L}")


@pytest.mark.parametrize("G", [1, 4])
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_rows_past_seq_len_never_matter(G, dtype):
    # the last resident page holds NaN patterns after the sequence's final token
    w = wl(Hq=2 * G, Hkv=2, dtype=dtype, seq_lens=[701, 333], tok_begin=[130, 5], tok_end=[701, 333], seed=5)
    run_and_check(w, poison_tail=True)


@pytest.mark.parametrize("G", [1, 8])
def test_outlier_tokens(G):
    w = wl(B=1, Hq=G, Hkv=1, seq_lens=[3000], tok_begin=[1200], tok_end=[3000], outlier_frac=0.01, chunk_tokens=256, seed=9)
    run_and_check(w)


def test_all_slices_empty_gives_zero_and_minus_inf():
    w = wl(seq_lens=[50, 60], tok_begin=[50, 0], tok_end=[50, 0])
    prob = DeviceProblem(w, DEV)
    prob.partial()
    prob.merge([])
    torch.cuda.synchronize()
    assert (prob.out == 0).all() and torch.isinf(prob.lse).all() and (prob.lse < 0).all()
    assert torch.isinf(prob.m_part).all() and (prob.l_part == 0).all() and (prob.o_part == 0).all()


def test_extra_chunk_slots_are_neutral():
    w = wl()
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    NC = prob.NC + 3
    prob.NC = NC
    prob.desc = prob.make_desc(w.chunk_tokens, NC)
    prob.o_part = torch.full((w.B, w.Hq, NC, w.D), 7.0, device=DEV)
    prob.m_part = torch.full((w.B, w.Hq, NC), 7.0, device=DEV)
    prob.l_part = torch.full((w.B, w.Hq, NC), 7.0, device=DEV)
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    n1 = w.chunk_grid(1)[1]
    assert torch.isinf(prob.m_part[1, :, n1:]).all() and (prob.l_part[1, :, n1:] == 0).all()
    assert (prob.o_part[1, :, n1:] == 0).all()
    check_output(prob.out, prob.lse, ref.out, ref.lse)


# ---- split invariance and reproducibility on the GPU -----------------------------------------------------

@pytest.mark.parametrize("G", [1, 4])
def test_merged_result_is_invariant_to_chunking_and_bit_reproducible(G):
    w = wl(Hq=2 * G, Hkv=2, seq_lens=[2100, 900], tok_begin=[400, 100], tok_end=[2100, 900])
    ref = OracleRef(w)
    outs = []
    for chunk in (64, 128, 512, 2048):
        wc = dataclasses.replace(w, chunk_tokens=chunk)
        prob = DeviceProblem(wc, DEV)
        host = ref.host_partials_device(DEV)
        prob.step(host)
        torch.cuda.synchronize()
        check_output(prob.out, prob.lse, ref.out, ref.lse, f"chunk {chunk}")
        first = (prob.out.clone(), prob.lse.clone(), prob.o_part.clone())
        prob.step(host)
        torch.cuda.synchronize()
        assert torch.equal(prob.out, first[0]) and torch.equal(prob.lse, first[1]) and torch.equal(prob.o_part, first[2])
        outs.append(prob.out.double().cpu().numpy())
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() <= 2e-3


def test_merge_is_invariant_to_how_host_partials_are_split():
    w = wl(B=1, Hq=4, Hkv=1, seq_lens=[1200], tok_begin=[800], tok_end=[1200])
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    prob.partial()
    # host slice [0, 800) as 1, 2 or 5 partials in a single source, or as separate sources
    from oracle import hg_oracle as O
    for cuts in ([0, 800], [0, 300, 800], [0, 100, 101, 400, 799, 800]):
        parts = [O.chunked_partials(ref.q, ref.K, ref.V, w.dtype, [a], [b], 0, 1) for a, b in zip(cuts[:-1], cuts[1:])]
        m = np.concatenate([p[0] for p in parts], axis=2); l = np.concatenate([p[1] for p in parts], axis=2)
        o = np.concatenate([p[2] for p in parts], axis=2)
        src = tuple(torch.from_numpy(x).float().to(DEV) for x in (o, m, l))
        prob.merge([src])
        torch.cuda.synchronize()
        check_output(prob.out, prob.lse, ref.out, ref.lse, f"one source, cuts {cuts}")
        if len(parts) <= 5:
            srcs = [tuple(torch.from_numpy(x).float().to(DEV) for x in (p[2], p[0], p[1])) for p in parts]
            prob.merge(srcs)
            torch.cuda.synchronize()
            check_output(prob.out, prob.lse, ref.out, ref.lse, f"{len(srcs)} sources")


# ---- the fused entry points ---------------------------------------------------------------------------------

@pytest.mark.parametrize("G", [1, 4])
def test_decode_and_decode_host_match_partial_plus_merge(G):
    w = wl(Hq=2 * G, Hkv=2)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    host_dev = ref.host_partials_device(DEV)
    prob.step(host_dev)
    torch.cuda.synchronize()
    want_out, want_lse = prob.out.clone(), prob.lse.clone()

    nbytes = pkg.hg_attn_workspace_bytes(prob.desc, 2)
    ws = torch.empty(nbytes, dtype=torch.uint8, device=DEV)
    out = torch.empty_like(prob.out); lse = torch.empty_like(prob.lse)
    pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, host_dev,
                       out, lse, ws, prob.desc)
    torch.cuda.synchronize()
    assert torch.equal(out, want_out) and torch.equal(lse, want_lse)

    pin = lambda t: t.cpu().pin_memory()
    host_pinned = [tuple(pin(x) for x in src) for src in host_dev]
    out_h = torch.empty(prob.out.shape, dtype=torch.float32).pin_memory()
    lse_h = torch.empty(prob.lse.shape, dtype=torch.float32).pin_memory()
    pkg.hg_attn_decode_host(pin(prob.q), prob.kv["k"], prob.kv["v"], pin(prob.seq_lens), pin(prob.tok_begin),
                            pin(prob.tok_end), host_pinned, out_h, lse_h, ws, prob.desc)
    torch.cuda.synchronize()
    assert torch.equal(out_h, want_out.cpu()) and torch.equal(lse_h, want_lse.cpu())
    check_output(out_h, lse_h, ref.out, ref.lse)


@pytest.mark.parametrize("pinned", [True, False])
def test_decode_host_with_a_host_source_of_several_partials(pinned):
    """The workspace is sized by the number of host PARTIALS (the sum of the sources' nc), not of sources: one host
    source that carries the host-held prefix as three chunk partials needs room for three."""
    from oracle import hg_oracle as O
    w = wl(Hq=8, Hkv=2, seq_lens=[900, 411], tok_begin=[300, 130], tok_end=[900, 411])
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    m, l, o = O.chunked_partials(ref.q, ref.K, ref.V, w.dtype, [0, 0], w.tok_begin, 128, 3)     # prefix in 128-token chunks
    to = (lambda a: torch.from_numpy(a).float().pin_memory()) if pinned else (lambda a: torch.from_numpy(a).float())
    host_h = [(to(o), to(m), to(l))]
    need = pkg.hg_attn_workspace_bytes(prob.desc, 3)
    assert need > pkg.hg_attn_workspace_bytes(prob.desc, 1)
    ws = torch.empty(need, dtype=torch.uint8, device=DEV)
    pin = (lambda t: t.cpu().pin_memory()) if pinned else (lambda t: t.cpu())
    out_h, lse_h = pin(torch.empty_like(prob.out)), pin(torch.empty_like(prob.lse))
    pkg.hg_attn_decode_host(pin(prob.q), prob.kv["k"], prob.kv["v"], pin(prob.seq_lens), pin(prob.tok_begin),
                            pin(prob.tok_end), host_h, out_h, lse_h, ws, prob.desc)
    torch.cuda.synchronize()
    check_output(out_h, lse_h, ref.out, ref.lse, "host source with nc = 3")
    if not pinned:      # the staged form checks the size it was given against what this source needs
        small = torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, 1), dtype=torch.uint8, device=DEV)
        with pytest.raises(hg.HgError) as e:
            pkg.hg_attn_decode_host(pin(prob.q), prob.kv["k"], prob.kv["v"], pin(prob.seq_lens), pin(prob.tok_begin),
                                    pin(prob.tok_end), host_h, out_h, lse_h, small, prob.desc)
        assert e.value.status == hg.HG_ERR_WORKSPACE


@pytest.mark.parametrize("how", ["pinned", "pageable", "pinned_copies", "mixed", "unaligned"])
def test_decode_host_paths_agree(how):
    """Pinned host buffers are read and written by the kernels in place; pageable ones (or a mix, or a
    host partial the merge cannot read with 16-byte loads) go through staged copies.  Same bits either way."""
    w = wl(Hq=8, Hkv=2, seq_lens=[900, 411], tok_begin=[77, 0], tok_end=[900, 300])
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    host_dev = ref.host_partials_device(DEV)
    prob.step(host_dev)
    torch.cuda.synchronize()
    if how == "pinned_copies":
        prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, tune=hg.HG_TUNE_NO_HOST_DIRECT)
    pin = (lambda t: t.cpu()) if how == "pageable" else (lambda t: t.cpu().pin_memory())
    host_h = [tuple(pin(x) for x in src) for src in host_dev]
    if how == "mixed":
        host_h[1] = tuple(x.cpu() for x in host_dev[1])          # one pageable buffer sends the whole call to copies
    if how == "unaligned":
        o, m, l = host_h[0]
        shifted = torch.empty(o.numel() + 1, dtype=torch.float32).pin_memory()
        shifted[1:].copy_(o.reshape(-1))
        host_h[0] = (shifted[1:].view(o.shape), m, l)
        assert host_h[0][0].data_ptr() % 16 == 4
    out_h = torch.full(prob.out.shape, float("nan"), dtype=torch.float32)
    lse_h = torch.full(prob.lse.shape, float("nan"), dtype=torch.float32)
    if how != "pageable":
        out_h, lse_h = out_h.pin_memory(), lse_h.pin_memory()
    ws = torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, 2), dtype=torch.uint8, device=DEV)
    q_h, sl_h, tb_h, te_h = pin(prob.q), pin(prob.seq_lens), pin(prob.tok_begin), pin(prob.tok_end)
    for _ in range(2):
        pkg.hg_attn_decode_host(q_h, prob.kv["k"], prob.kv["v"], sl_h, tb_h, te_h, host_h, out_h, lse_h, ws, prob.desc)
        torch.cuda.synchronize()
    assert torch.equal(out_h, prob.out.cpu()) and torch.equal(lse_h, prob.lse.cpu())
    check_output(out_h, lse_h, ref.out, ref.lse, how)
    # the same call with its arguments marshalled once
    call = pkg.prepare_decode_host(q_h, prob.kv["k"], prob.kv["v"], sl_h, tb_h, te_h, host_h, out_h, lse_h, ws, prob.desc)
    out_h.fill_(float("nan"))
    call()
    torch.cuda.synchronize()
    assert torch.equal(out_h, prob.out.cpu()) and torch.equal(lse_h, prob.lse.cpu())


# ---- the read probe moves exactly the slice's bytes -------------------------------------------------------------

@pytest.mark.parametrize("layout", ["HND", "NHD"])
def test_read_probe_checksum_is_the_xor_of_the_slice(layout):
    w = wl(layout=layout, seq_lens=[700, 333], tok_begin=[130, 5], tok_end=[700, 290])
    prob = DeviceProblem(w, DEV)
    sink = torch.zeros(w.B, w.Hkv, prob.NC, dtype=torch.int32, device=DEV)
    pkg.hg_kv_read_probe(prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, sink, prob.desc)
    torch.cuda.synchronize()
    got = sink.cpu().numpy().view(np.uint32)
    for b in range(w.B):
        for g in range(w.Hkv):
            for c in range(prob.NC):
                lo, hi = w.chunk_range(b, c)
                want = np.uint32(0)
                if hi > lo:
                    for which in ("k", "v"):
                        words = bits(w.kv_rows(which, b, g, lo, hi)).reshape(-1).view(np.uint32)
                        want ^= np.bitwise_xor.reduce(words)
                assert got[b, g, c] == want, (b, g, c)


def partials_over_index_sets(w, prob, keep):
    """Oracle chunk partials when only the tokens `keep(b, t)` of each slice count."""
    from oracle import hg_oracle as O
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    NC, D = prob.NC, w.D
    rm = np.full((w.B, w.Hq, NC), -np.inf); rl = np.zeros((w.B, w.Hq, NC)); ro = np.zeros((w.B, w.Hq, NC, D))
    for b in range(w.B):
        for c in range(w.chunk_grid(b)[1]):
            lo, hi = w.chunk_range(b, c)
            idx = [t for t in range(lo, hi) if keep(b, t)]
            for h in range(w.Hq):
                g = h // w.G
                rm[b, h, c], rl[b, h, c], ro[b, h, c] = O.partial(q[b, h], np.ascontiguousarray(K[b, :, g]),
                                                                   np.ascontiguousarray(V[b, :, g]), w.dtype, idx=idx)
    return rm, rl, ro


@pytest.mark.parametrize("G,page", [(1, 16), (4, 16), (1, 64), (8, 32)])
def test_bad_page_id_is_reported_and_its_tokens_left_out(G, page):
    """A block-table entry outside the pool is never dereferenced: the call is flagged and the partials are those
    of the slice without that page's tokens (rows of the box that was not loaded must not leak stale data)."""
    w = wl(Hq=2 * G, Hkv=2, page_size=page, chunk_tokens=128, seed=90 + G)
    prob = DeviceProblem(w, DEV)
    # fill the ring with another call first, so that a skipped box would expose stale rows
    prob.partial()
    table = prob.kv["block_table"].clone()
    bad = w.tok_begin[0] // w.page_size + 3
    table[0, bad] = prob.kv["num_pages"] + 5
    whole_chunk = [pg for pg in range(w.max_pages) if pg * page >= 256 and (pg + 1) * page <= 384]   # a chunk with no page left
    for pg in whole_chunk:
        table[1, pg] = -7
    prob.kv = dict(prob.kv, block_table=table)
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC)
    prob.partial()
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_BAD_PAGE

    def keep(b, t):
        pg = t // page
        return not ((b == 0 and pg == bad) or (b == 1 and pg in whole_chunk))

    rm, rl, ro = partials_over_index_sets(w, prob, keep)
    assert np.isinf(rm[1, :, (256 - (w.tok_begin[1] // 128) * 128) // 128]).all()        # that chunk became an empty partial
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D), "bad page")


@pytest.mark.parametrize("G", [1, 4])
@pytest.mark.parametrize("persistent", [True, False])
def test_slice_beyond_the_block_table_is_cut_and_reported(G, persistent):
    """seq_lens and tok_end live on the device, so the host cannot check them against max_pages: a slice that reaches
    past the table's last page is cut there, the call is flagged, and the partials are those of the cut slice."""
    w = wl(Hq=2 * G, Hkv=2, seed=95 + G)
    prob = DeviceProblem(w, DEV)
    short = 35                                               # pages the table row is cut to: 560 tokens < 700
    assert short * w.page_size < w.tok_end[0] and short * w.page_size > w.tok_end[1]
    table = prob.kv["block_table"][:, :short].contiguous()
    prob.kv = dict(prob.kv, block_table=table, max_pages=short)
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, tune=0 if persistent else hg.HG_TUNE_NO_PERSISTENT)
    prob.partial()
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_RANGE
    rm, rl, ro = partials_over_index_sets(w, prob, lambda b, t: t < short * w.page_size)
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D), "beyond table")


# ---- bit patterns the seeded generator never produces -----------------------------------------------------------

@pytest.mark.parametrize("G,dtype", [(1, "f16"), (1, "bf16"), (4, "f16"), (8, "bf16")])
def test_subnormals_zeros_and_large_values_in_the_cache(G, dtype):
    """The generator draws from a table of normal quantiles: no subnormal, no signed zero, nothing beyond 4.4 sigma.  Here a
    tenth of the resident K and V elements and a few q elements are overwritten with such patterns (subnormals of either
    sign, -0, the smallest normals, values up to +-48); the oracle decodes the same bits exactly, and the GPU path - the
    fp32 unpacking of the one-head kernel as well as the tensor-core operands of the group-query one - must agree."""
    from oracle import hg_oracle as O
    w = wl(B=2, Hq=2 * G, Hkv=2, D=128, dtype=dtype, seq_lens=[700, 333], tok_begin=[130, 5], tok_end=[700, 290], seed=120 + G)
    prob = DeviceProblem(w, DEV)
    gen = torch.Generator(device=DEV).manual_seed(5)
    if dtype == "f16":
        special = [0x0001, 0x8001, 0x03FF, 0x83FF, 0x8000, 0x0400, 0x8400, 0x5200, 0xD200, 0x4E00]   # subnormals, -0, 2^-14, +-48, 24
    else:
        special = [0x0001, 0x8001, 0x007F, 0x807F, 0x8000, 0x0080, 0x8080, 0x4240, 0xC240, 0x41C0]   # the same for bf16
    pat = torch.tensor(special, dtype=torch.int32, device=DEV)
    for pool in (prob.kv["k"], prob.kv["v"], prob.q):
        flat = pool.view(torch.int16).view(-1)
        hit = torch.rand(flat.numel(), device=DEV, generator=gen) < (0.1 if pool is not prob.q else 0.02)
        pick = pat[torch.randint(0, len(special), (flat.numel(),), device=DEV, generator=gen)]
        flat[hit] = pick[hit].to(torch.int16)
    # the logical cache as the block table maps it (pages of the slice only; the rest is never read)
    ps, table = w.page_size, prob.kv["block_table"].cpu()
    K = np.zeros((w.B, w.max_len, w.Hkv, w.D), dtype=np.uint16); V = np.zeros_like(K)
    kp, vp = bits(prob.kv["k"]), bits(prob.kv["v"])                         # [pages][Hkv][ps][D]
    for b in range(w.B):
        for pg in range(w.tok_begin[b] // ps, -(-w.tok_end[b] // ps)):
            n = min(ps, w.max_len - pg * ps)
            K[b, pg * ps: pg * ps + n] = kp[int(table[b, pg])].transpose(1, 0, 2)[:n]
            V[b, pg * ps: pg * ps + n] = vp[int(table[b, pg])].transpose(1, 0, 2)[:n]
    q = bits(prob.q)
    prob.step([])
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    rm, rl, ro = O.chunked_partials(q, K, V, dtype, w.tok_begin, w.tok_end, w.chunk_tokens, prob.NC)
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D), "special values")
    ref_out, ref_lse = O.full_batch(q, K, V, dtype, w.tok_begin, w.tok_end)
    check_output(prob.out, prob.lse, ref_out, ref_lse, "special values")
    assert np.abs(ref_out).max() > 1.0          # the large values do reach the output


# ---- schedules: persistent-dynamic, persistent-static and one-CTA-per-item give the same bits --------------------

@pytest.mark.parametrize("G", [1, 4])
def test_result_does_not_depend_on_the_schedule(G):
    w = wl(B=3, Hq=2 * G, Hkv=2, seq_lens=[2100, 900, 333], tok_begin=[400, 100, 333], tok_end=[2100, 900, 333],
           chunk_tokens=128)
    ref = OracleRef(w)
    results = []
    for env in ({}, {"tune": hg.HG_TUNE_NO_DYNAMIC}, {"tune": hg.HG_TUNE_NO_PERSISTENT}, {"tune_stages": 2},
                {"tune_ctas_per_sm": 1, "tune_stages": 5}, {"tune": hg.HG_TUNE_NO_PDL}, {"tune": hg.HG_TUNE_NO_SPEC_PREFETCH}):
        prob = DeviceProblem(w, DEV)
        prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, **env)
        prob.step(ref.host_partials_device(DEV))
        torch.cuda.synchronize()
        assert int(prob.status.item()) == hg.HG_DEV_OK
        check_output(prob.out, prob.lse, ref.out, ref.lse, str(env))
        results.append((prob.o_part.clone(), prob.m_part.clone(), prob.l_part.clone(), prob.out.clone()))
    for r in results[1:]:
        for a, b in zip(results[0], r):
            assert torch.equal(a, b)


def test_a_ring_that_does_not_fit_shared_memory_is_refused_and_the_next_call_works():
    w = wl(B=2, Hq=4, Hkv=2, seq_lens=[900, 333], tok_begin=[100, 0], tok_end=[900, 333], chunk_tokens=128)
    prob = DeviceProblem(w, DEV)
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, tune_stages=8)         # 8 x 34 KB: more than an SM has
    with pytest.raises(hg.HgError) as e:
        prob.partial()
    assert e.value.status == hg.HG_ERR_CUDA
    torch.cuda.synchronize()                                                      # no error is left behind
    run_and_check(w)


@pytest.mark.parametrize("G", [1, 8])
def test_every_call_leaves_the_work_counter_at_zero(G):
    """More items than resident CTAs, so the counter hands them out.  The last CTA to stop drawing clears both
    words: with HG_FLAG_COUNTER_CLEAN the next call runs without any clearing in front of it (and may start as a
    programmatic dependent) and gives the same bits as a call that cleared the counter itself."""
    w = wl(B=6, Hq=4 * G, Hkv=4, seq_lens=[6000] * 6, tok_begin=[100] * 6, tok_end=[6000] * 6, chunk_tokens=64, seed=70 + G)
    assert sum(w.chunk_grid(b)[1] for b in range(w.B)) * w.Hkv > 2 * 296
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    assert prob.sched.tolist() == [0, 0]
    want = (prob.o_part.clone(), prob.m_part.clone(), prob.l_part.clone(), prob.out.clone(), prob.lse.clone())
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, flags=hg.HG_FLAG_COUNTER_CLEAN)
    for _ in range(3):
        for t in (prob.o_part, prob.m_part, prob.l_part, prob.out, prob.lse):
            t.fill_(float("nan"))
        prob.step(ref.host_partials_device(DEV))        # back to back: partial, merge, partial, ...
    torch.cuda.synchronize()
    assert prob.sched.tolist() == [0, 0] and int(prob.status.item()) == hg.HG_DEV_OK
    for a, b in zip(want, (prob.o_part, prob.m_part, prob.l_part, prob.out, prob.lse)):
        assert torch.equal(a, b)
    check_output(prob.out, prob.lse, ref.out, ref.lse)
    # the fused entry point keeps its counter in the workspace: with the flag, a zero-filled workspace serves call after call
    ws = torch.zeros(pkg.hg_attn_workspace_bytes(prob.desc, 2), dtype=torch.uint8, device=DEV)
    for _ in range(3):
        out, lse = torch.full_like(prob.out, float("nan")), torch.full_like(prob.lse, float("nan"))
        pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                           ref.host_partials_device(DEV), out, lse, ws, prob.desc)
        torch.cuda.synchronize()
        assert torch.equal(out, want[3]) and torch.equal(lse, want[4])


def test_without_a_work_counter_items_are_dealt_round_robin():
    w = wl(Hq=8, Hkv=2)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    prob.sched = None
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC)
    assert not prob.desc.sched_counter
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    check_output(prob.out, prob.lse, ref.out, ref.lse)


# ---- shapes beyond what the persistent schedule keeps in shared memory fall back to one CTA per item ------------

@pytest.mark.parametrize("B", [530, 1024, 1030])
def test_large_batches(B):
    # up to 1024 sequences the in-kernel item scan (every thread several sequences) feeds the persistent schedule;
    # beyond that the same kernel runs with one CTA per item
    lens = [40 + (7 * i) % 150 for i in range(B)]
    tb = [(3 * i) % 30 for i in range(B)]
    w = wl(B=B, Hq=2, Hkv=1, D=64, seq_lens=lens, tok_begin=tb, tok_end=lens, chunk_tokens=64, seed=77)
    run_and_check(w)


def test_chunks_with_many_pages_use_the_per_item_grid():
    # 8192-token chunks of 16-token pages: 512 page ids per chunk, beyond the double-buffered page list
    w = wl(B=1, Hq=4, Hkv=1, seq_lens=[9000], tok_begin=[100], tok_end=[9000], chunk_tokens=8192, seed=78)
    run_and_check(w)


@pytest.mark.parametrize("G,layout", [(1, "HND"), (4, "HND"), (4, "NHD")])
def test_pages_above_four_gib_in_the_pool(G, layout):
    # pools of 6 GiB each whose live pages are the last ones: page offsets need more than 32 bits, in bytes and in
    # elements; everything below the live pages is uninitialised memory that no box may touch
    w = wl(Hq=2 * G, Hkv=2, page_size=64, layout=layout, chunk_tokens=256, seq_lens=[1500, 777], tok_begin=[70, 0],
           tok_end=[1500, 700], seed=79)
    small = w.build_device_kv(DEV)
    page_elems = small["page_stride"]
    total_pages = (6 << 30) // (2 * page_elems)
    shift = total_pages - small["num_pages"]
    assert shift * page_elems > 2**31
    kv = dict(small)
    for which in ("k", "v"):
        big = torch.empty((total_pages,) + tuple(small[which].shape[1:]), dtype=small[which].dtype, device=DEV)
        big[:64].fill_(float("nan"))
        big[shift:] = small[which]
        kv[which] = big
    table = small["block_table"]
    kv["block_table"] = torch.where(table >= 0, table + shift, table)
    kv["num_pages"] = total_pages
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV, kv=kv)
    prob.partial()
    prob.merge(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    rm, rl, ro = ref.chunk_partials(w.chunk_tokens, prob.NC)
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D))
    check_output(prob.out, prob.lse, ref.out, ref.lse)
    # the same through the read probe: the checksum of exactly the slice's bits
    small_prob = DeviceProblem(w, DEV, kv=small)
    sinks = []
    for pr in (prob, small_prob):
        sink = torch.zeros(w.B, w.Hkv, pr.NC, dtype=torch.int32, device=DEV)
        pkg.hg_kv_read_probe(pr.kv["k"], pr.kv["v"], pr.seq_lens, pr.tok_begin, pr.tok_end, sink, pr.desc)
        sinks.append(sink)
    torch.cuda.synchronize()
    assert torch.equal(sinks[0], sinks[1])
    del prob, kv, big
    torch.cuda.empty_cache()


# ---- bounded waits: a stalled pipeline ends with a status code, not a hang -----------------------------------------

@pytest.mark.parametrize("G", [1, 4])
def test_stalled_loader_times_out_with_a_status_and_the_context_stays_usable(G):
    import time
    w = wl(B=1, Hq=2 * G, Hkv=2, seq_lens=[300], tok_begin=[0], tok_end=[300])
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    prob.desc.flags = hg.HG_FLAG_TEST_STALL          # nothing ever fills a stage: every consumer wait must run out
    torch.cuda.synchronize()
    t0 = time.time()
    prob.partial()
    torch.cuda.synchronize()
    dt = time.time() - t0
    assert int(prob.status.item()) == hg.HG_DEV_WAIT_TIMEOUT
    assert 1.0 < dt < 30.0
    # while the word is set, later launches return at once instead of queueing behind a broken pipeline
    prob.desc.flags = 0
    t0 = time.time()
    prob.partial()
    torch.cuda.synchronize()
    assert time.time() - t0 < 1.0 and int(prob.status.item()) == hg.HG_DEV_WAIT_TIMEOUT
    # cleared: the same context computes correct results again
    prob.status.zero_()
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    check_output(prob.out, prob.lse, ref.out, ref.lse)


# ---- the decode call sequence can be captured in a CUDA graph and replayed ------------------------------------------

@pytest.mark.parametrize("G", [1, 4])
def test_decode_replays_from_a_cuda_graph(G):
    w = wl(Hq=2 * G, Hkv=2)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    host = ref.host_partials_device(DEV)
    ws = torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, 2), dtype=torch.uint8, device=DEV)
    out = torch.empty_like(prob.out); lse = torch.empty_like(prob.lse)
    call = lambda: pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                                      host, out, lse, ws, prob.desc)
    call()                                            # warm up outside the capture (first-use set-up of the kernels)
    torch.cuda.synchronize()
    want_out, want_lse = out.clone(), lse.clone()
    side = torch.cuda.Stream()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        with torch.cuda.graph(graph, stream=side):
            call()
    for _ in range(3):
        out.fill_(float("nan")); lse.fill_(float("nan"))
        graph.replay()
        torch.cuda.synchronize()
        assert torch.equal(out, want_out) and torch.equal(lse, want_lse)
    # device-resident ranges: the same graph follows a changed slice without re-capture
    prob.tok_begin += 64
    ref2 = OracleRef(dataclasses.replace(w, tok_begin=[t + 64 for t in w.tok_begin]))
    for dst, src in zip(host, ref2.host_partials_device(DEV)):
        for a, b in zip(dst, src):
            a.copy_(b)
    graph.replay()
    torch.cuda.synchronize()
    check_output(out, lse, ref2.out, ref2.lse, "replayed on a moved slice")


# ---- seeded random sweep over everything at once ---------------------------------------------------------------------

@pytest.mark.parametrize("seed", range(24))
def test_random_shapes(seed):
    rng = np.random.default_rng(1000 + seed)
    B = int(rng.integers(1, 6))
    Hkv = int(rng.choice([1, 2, 3]))
    G = int(rng.choice([1, 1, 2, 4, 5, 8, 9, 16]))
    D = int(rng.choice([64, 128]))
    page = int(rng.choice([16, 32, 64, 128]))
    layout, paged = [("HND", True), ("NHD", True), ("NHD", False)][int(rng.integers(0, 3))]
    chunk = int(rng.choice([64, 128, 256, 512]))
    chunk = max(chunk, page)
    lens = [int(rng.integers(1, 1400)) for _ in range(B)]
    tb, te = [], []
    for L in lens:
        kind = rng.integers(0, 5)
        if kind == 0:
            a = e = int(rng.integers(0, L + 1))                   # empty slice
        elif kind == 1:
            a, e = 0, L                                           # whole sequence on the GPU
        else:
            a = int(rng.integers(0, L)); e = int(rng.integers(a, L + 1))
        tb.append(a); te.append(e)
    w = W.AttnWorkload(f"rand{seed}", B, Hkv * G, Hkv, D, str(rng.choice(["f16", "bf16"])), lens, tb, te, page_size=page,
                       layout=layout, paged=paged, chunk_tokens=chunk, seed=2000 + seed,
                       sigma_kv=float(rng.choice([0.5, 1.0, 2.0])), outlier_frac=float(rng.choice([0.0, 0.02])))
    run_and_check(w, poison_tail=bool(rng.integers(0, 2)), what=repr(w))


@pytest.mark.parametrize("dynamic", ["1", "0"])
@pytest.mark.parametrize("seed", range(5))
def test_random_shapes_with_many_items_per_cta(seed, dynamic):
    """Several hundred to a couple of thousand work items: every resident CTA takes several, so the ring runs
    across item boundaries, the look-ahead of item indices and page ids is in play, and (dynamic) the counter."""
    rng = np.random.default_rng(50000 + seed)
    B = int(rng.integers(4, 9))
    Hkv = int(rng.choice([4, 8]))
    G = int(rng.choice([1, 2, 4, 8]))
    D = int(rng.choice([64, 128]))
    page = int(rng.choice([16, 64]))
    chunk = max(int(rng.choice([64, 128])), page)
    layout, paged = [("HND", True), ("NHD", True), ("NHD", False)][int(rng.integers(0, 3))]
    lens = [int(rng.integers(4000, 8000)) for _ in range(B)]
    tb = [int(rng.integers(0, L // 4)) for L in lens]
    te = [int(rng.integers(3 * L // 4, L + 1)) for L in lens]
    w = W.AttnWorkload(f"many{seed}", B, Hkv * G, Hkv, D, str(rng.choice(["f16", "bf16"])), lens, tb, te, page_size=page,
                       layout=layout, paged=paged, chunk_tokens=chunk, seed=7000 + seed)
    assert sum(w.chunk_grid(b)[1] for b in range(B)) * Hkv > 296
    run_and_check(w, what=repr(w)[:200], tune=0 if dynamic == "1" else hg.HG_TUNE_NO_DYNAMIC)


# ---- a token set made of several ranges (Section 4.3's position-based choice: sinks + recent window) ----

@pytest.mark.parametrize("G", [1, 4])
def test_sinks_plus_recent_window_as_two_ranges(G):
    """Two calls over disjoint ranges of the same pool, merged as two sources, give attention over
    exactly the union of the ranges."""
    from oracle import hg_oracle as O
    L, sinks, window = [1500, 777], 4, [600, 130]
    w = wl(Hq=2 * G, Hkv=2, seq_lens=L, tok_begin=[0, 0], tok_end=L, chunk_tokens=256, seed=77)
    prob = DeviceProblem(w, DEV)
    parts = []
    for lo, hi in (([0, 0], [sinks, sinks]), ([l - n for l, n in zip(L, window)], L)):
        o, m, l = torch.empty_like(prob.o_part), torch.empty_like(prob.m_part), torch.empty_like(prob.l_part)
        hg.hg_attn_partial(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens,
                           torch.tensor(lo, dtype=torch.int32, device=DEV), torch.tensor(hi, dtype=torch.int32, device=DEV),
                           o, m, l, prob.desc)
        parts.append((o, m, l))
    hg.hg_attn_merge(parts, prob.out, prob.lse, prob.desc)
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    ref_out = np.empty((w.B, w.Hq, w.D)); ref_lse = np.empty((w.B, w.Hq))
    for b in range(w.B):
        idx = np.concatenate([np.arange(sinks), np.arange(L[b] - window[b], L[b])]).astype(np.int64)
        for h in range(w.Hq):
            g = h // G
            ref_out[b, h], ref_lse[b, h] = O.full(q[b, h], np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g]),
                                                   w.dtype, idx=idx)
    check_output(prob.out, prob.lse, ref_out, ref_lse, "sinks + window")


@pytest.mark.parametrize("G,page", [(1, 16), (4, 16), (8, 64)])
def test_selected_pages_through_a_compacted_block_table(G, page):
    """A page-granular token set (a Pre-QK^T choice of whole pages, say): the caller lists the chosen pages of each
    sequence in a block table of their own, in token order, and attends the range [0, pages * page_size) of that
    virtual sequence; the result is attention over exactly the chosen pages' tokens."""
    from oracle import hg_oracle as O
    L = [1500, 777]
    w = wl(Hq=2 * G, Hkv=2, page_size=page, seq_lens=L, tok_begin=[0, 0], tok_end=L, chunk_tokens=256, seed=83)
    prob = DeviceProblem(w, DEV)
    rng = np.random.default_rng(83)
    full_pages = [l // page for l in L]                      # the ragged last page stays out of the choice
    chosen = [np.sort(rng.choice(n, size=max(1, n // 3), replace=False)) for n in full_pages]
    chosen[1] = np.union1d(chosen[1], [0, full_pages[1] - 1])
    width = max(len(c) for c in chosen)
    table = torch.full((w.B, width), -1, dtype=torch.int32, device=DEV)
    for b, c in enumerate(chosen):
        table[b, :len(c)] = prob.kv["block_table"][b, torch.as_tensor(c, device=DEV)]
    n_tok = [len(c) * page for c in chosen]
    NC = (max(n_tok) + 255) // 256
    prob.kv = dict(prob.kv, block_table=table, max_pages=width)
    desc = prob.make_desc(256, NC)
    lens = torch.tensor(n_tok, dtype=torch.int32, device=DEV)
    o = torch.empty(w.B, w.Hq, NC, w.D, device=DEV); m = torch.empty(w.B, w.Hq, NC, device=DEV); l = torch.empty_like(m)
    hg.hg_attn_partial(prob.q, prob.kv["k"], prob.kv["v"], lens, torch.zeros_like(lens), lens, o, m, l, desc)
    hg.hg_attn_merge([(o, m, l)], prob.out, prob.lse, desc)
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    ref_out = np.empty((w.B, w.Hq, w.D)); ref_lse = np.empty((w.B, w.Hq))
    for b in range(w.B):
        idx = (chosen[b][:, None] * page + np.arange(page)[None, :]).reshape(-1).astype(np.int64)
        for h in range(w.Hq):
            g = h // G
            ref_out[b, h], ref_lse[b, h] = O.full(q[b, h], np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g]),
                                                   w.dtype, idx=idx)
    check_output(prob.out, prob.lse, ref_out, ref_lse, "selected pages")


@pytest.mark.parametrize("G", [1, 4])
def test_a_slice_longer_than_num_chunks_is_cut_to_its_first_chunks(G):
    """num_chunks bounds the work: tokens past the last chunk slot are not attended, and what is produced equals attention over the kept range."""
    C, keep = 128, 3
    w = wl(Hq=2 * G, Hkv=2, seq_lens=[900, 500], tok_begin=[70, 0], tok_end=[900, 200], chunk_tokens=C, seed=31)
    prob = DeviceProblem(w, DEV)
    assert prob.NC > keep
    prob.NC = keep
    prob.desc = prob.make_desc(C, keep)
    prob.o_part = torch.empty(w.B, w.Hq, keep, w.D, device=DEV)
    prob.m_part = torch.empty(w.B, w.Hq, keep, device=DEV)
    prob.l_part = torch.empty(w.B, w.Hq, keep, device=DEV)
    prob.step([])
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    kept_end = [min(te, (tb // C + keep) * C) for tb, te in zip(w.tok_begin, w.tok_end)]
    assert kept_end == [384, 200]
    w_cut = dataclasses.replace(w, tok_end=kept_end)
    ref = OracleRef(w_cut)
    rm, rl, ro = ref.chunk_partials(C, keep)
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D), "cut")
    from oracle import hg_oracle as O
    ref_out, ref_lse = O.full_batch(ref.q, ref.K, ref.V, w.dtype, w.tok_begin, kept_end)
    check_output(prob.out, prob.lse, ref_out, ref_lse, "cut")


def test_prepared_calls_are_the_same_calls():
    """prepare_partial / prepare_merge / DeviceProblem.prepare_step marshal once; the launches are identical."""
    w = wl(Hq=8, Hkv=2)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    host = ref.host_partials_device(DEV)
    prob.step(host)
    torch.cuda.synchronize()
    want_o, want_out, want_lse = prob.o_part.clone(), prob.out.clone(), prob.lse.clone()
    for t in (prob.o_part, prob.m_part, prob.l_part, prob.out, prob.lse):
        t.fill_(float("nan"))
    step = prob.prepare_step(host)
    for _ in range(3):
        step()
    torch.cuda.synchronize()
    assert torch.equal(prob.o_part, want_o) and torch.equal(prob.out, want_out) and torch.equal(prob.lse, want_lse)
    bad = pkg.prepare_merge([(prob.o_part, prob.m_part, prob.l_part)], prob.out, prob.lse,
                            prob.make_desc(w.chunk_tokens, prob.NC))
    bad()                                                   # a fresh description: still fine
    with pytest.raises(ValueError):
        pkg.prepare_partial(prob.q.cpu(), prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                            prob.o_part, prob.m_part, prob.l_part, prob.desc)


@pytest.mark.parametrize("D,G", [(128, 4), (64, 1)])
def test_many_short_rows_take_the_warp_per_row_merge(D, G):
    """A large batch of short sequences: thousands of (sequence, head) rows with a handful of partials each are
    merged a warp per row; same result as the CTA-per-row kernel up to summation order."""
    rng = np.random.default_rng(3)
    B, Hkv = 300, 2
    lens = [int(rng.integers(40, 330)) for _ in range(B)]
    tb = [int(rng.integers(0, L // 2)) for L in lens]
    te = [int(rng.integers(L // 2, L + 1)) for L in lens]
    te[5] = tb[5]                                              # an empty slice among them
    w = W.AttnWorkload("rows", B, Hkv * G * 4, Hkv, D, "f16", lens, tb, te, page_size=16, chunk_tokens=128, seed=41)
    assert w.B * w.Hq >= 2048
    prob, ref, _ = run_and_check(w)
    out_rows, lse_rows = prob.out.clone(), prob.lse.clone()
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, tune=hg.HG_TUNE_NO_MERGE_ROWS)
    prob.merge(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    check_output(prob.out, prob.lse, ref.out, ref.lse, "cta per row")
    assert (prob.out - out_rows).abs().max().item() <= 1e-5 * max(1.0, out_rows.abs().max().item())
    assert torch.equal(torch.isinf(prob.lse), torch.isinf(lse_rows))


@pytest.mark.parametrize("G", [9, 12, 16, 24])
def test_groups_of_more_than_8_heads_either_way(G):
    """Groups above 8 query heads run as items of 16 heads (two MMA head blocks sharing every tile read); the
    older form - one item per block of 8 - stays selectable.  Both match the oracle and each other."""
    w = wl(B=2, Hq=G, Hkv=1, D=128, dtype="bf16", seq_lens=[900, 300], tok_begin=[70, 0], tok_end=[900, 217],
           chunk_tokens=256, seed=300 + G, outlier_frac=0.01)
    prob, ref, _ = run_and_check(w)
    a_out, a_o = prob.out.clone(), prob.o_part.clone()
    prob2, _, _ = run_and_check(w, tune=hg.HG_TUNE_NO_GQA16)
    assert (prob2.out - a_out).abs().max().item() <= 1e-5 * max(1.0, a_out.abs().max().item())
    assert (prob2.o_part - a_o).abs().max().item() <= 1e-4 * max(1.0, a_o.abs().max().item())


@pytest.mark.parametrize("G", [1, 4, 16])
def test_explicit_scale_overrides_the_default(G):
    from oracle import hg_oracle as O
    w = wl(Hq=2 * G, Hkv=2, seed=500 + G)
    scale = 0.043
    prob = DeviceProblem(w, DEV)
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, scale=scale)
    prob.step([])
    torch.cuda.synchronize()
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    rm, rl, ro = O.chunked_partials(q, K, V, w.dtype, w.tok_begin, w.tok_end, w.chunk_tokens, prob.NC, scale=scale)
    check_partials(prob.o_part.reshape(-1, w.D), prob.m_part.reshape(-1), prob.l_part.reshape(-1),
                   rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, w.D), "scale")
    ref_out, ref_lse = O.full_batch(q, K, V, w.dtype, w.tok_begin, w.tok_end, scale=scale)
    check_output(prob.out, prob.lse, ref_out, ref_lse, "scale")
    # and it is not the default
    d_out, _ = O.full_batch(q, K, V, w.dtype, w.tok_begin, w.tok_end)
    assert np.abs(d_out - ref_out).max() > 1e-2


@pytest.mark.parametrize("G", [1, 4])
def test_ranges_reaching_outside_the_sequence_are_clipped(G):
    """tok_begin below 0 and tok_end above seq_len mean "from the start" and "to the end": rows past seq_len are never
    attended even when the caller's range covers them."""
    w = wl(Hq=2 * G, Hkv=2, seq_lens=[700, 333], tok_begin=[130, 0], tok_end=[700, 333], seed=61)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV, poison_tail=True)
    prob.tok_begin = torch.tensor([130, -7], dtype=torch.int32, device=DEV)
    prob.tok_end = torch.tensor([700 + 500, 333 + 1], dtype=torch.int32, device=DEV)
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK
    check_output(prob.out, prob.lse, ref.out, ref.lse, "clipped")


def test_two_streams_with_their_own_workspaces_do_not_disturb_each_other():
    """Two decode loops on two streams, each with its own workspace (and so its own work counter), interleaved
    launch by launch: every result is the one the loop gets alone.  (No launch waits for another.)"""
    ws_list, probs, wants, outs = [], [], [], []
    for i, G in enumerate((1, 4)):
        w = wl(Hq=8 * G, Hkv=8, seq_lens=[3000, 1777], tok_begin=[100, 0], tok_end=[3000, 1700], chunk_tokens=64, seed=700 + i)
        assert sum(w.chunk_grid(b)[1] for b in range(w.B)) * w.Hkv > 296      # more items than resident CTAs: the counter is in use
        prob = DeviceProblem(w, DEV)
        prob.step([])
        torch.cuda.synchronize()
        probs.append(prob)
        wants.append((prob.out.clone(), prob.lse.clone()))
        ws_list.append(torch.empty(pkg.hg_attn_workspace_bytes(prob.desc, 0), dtype=torch.uint8, device=DEV))
        outs.append((torch.empty_like(prob.out), torch.empty_like(prob.lse)))
    streams = [torch.cuda.Stream(device=DEV) for _ in probs]
    torch.cuda.synchronize()
    for _ in range(10):
        for prob, ws, (out, lse), st in zip(probs, ws_list, outs, streams):
            pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end, [], out, lse,
                               ws, prob.desc, stream=st)
    torch.cuda.synchronize()
    for prob, (out, lse), (want_out, want_lse) in zip(probs, outs, wants):
        assert int(prob.status.item()) == hg.HG_DEV_OK
        assert torch.equal(out, want_out) and torch.equal(lse, want_lse)


@pytest.mark.parametrize("G", [1, 4])
def test_sparse_empty_slots_for_mixed_batches(G):
    """A batch of one long and several short sequences: num_chunks follows the long one.  With HG_FLAG_SPARSE_EMPTY
    the short sequences' unused slots get m = -inf and l = 0 and their o rows are not touched; the merge never
    reads them.  hg_attn_decode works that way by itself."""
    lens = [2500, 90, 130, 64, 300]
    w = wl(B=5, Hq=2 * G, Hkv=2, seq_lens=lens, tok_begin=[0, 10, 0, 0, 37], tok_end=lens, chunk_tokens=128, seed=88)
    ref = OracleRef(w)
    prob = DeviceProblem(w, DEV)
    prob.desc = prob.make_desc(w.chunk_tokens, prob.NC, flags=hg.HG_FLAG_SPARSE_EMPTY)
    prob.o_part.fill_(float("nan")); prob.m_part.fill_(7.0); prob.l_part.fill_(7.0)
    prob.step(ref.host_partials_device(DEV))
    torch.cuda.synchronize()
    check_output(prob.out, prob.lse, ref.out, ref.lse, "sparse")
    for b in range(1, w.B):
        n = w.chunk_grid(b)[1]
        assert n < prob.NC
        assert torch.isinf(prob.m_part[b, :, n:]).all() and (prob.l_part[b, :, n:] == 0).all()
        assert torch.isnan(prob.o_part[b, :, n:]).all()                    # left alone
        assert not torch.isnan(prob.o_part[b, :, :n]).any()
    ws = torch.full((pkg.hg_attn_workspace_bytes(prob.desc, 2),), 0xFF, dtype=torch.uint8, device=DEV)   # NaN patterns
    out, lse = torch.empty_like(prob.out), torch.empty_like(prob.lse)
    plain = prob.make_desc(w.chunk_tokens, prob.NC)
    pkg.hg_attn_decode(prob.q, prob.kv["k"], prob.kv["v"], prob.seq_lens, prob.tok_begin, prob.tok_end,
                       ref.host_partials_device(DEV), out, lse, ws, plain)
    torch.cuda.synchronize()
    assert torch.equal(out, prob.out) and torch.equal(lse, prob.lse)


def test_the_readme_decode_flow():
    """The dozen lines of the README: suggest a chunk size, describe the pool by its tensor strides, decode."""
    G = 4
    w = wl(Hq=2 * G, Hkv=2, seq_lens=[1900, 777], tok_begin=[300, 0], tok_end=[1900, 700], seed=404)
    ref = OracleRef(w)
    kv = w.build_device_kv(DEV)
    k_pool, v_pool, block_table = kv["k"], kv["v"], kv["block_table"]
    assert k_pool.shape == (kv["num_pages"], w.Hkv, w.page_size, w.D)
    chunk = pkg.hg_attn_suggest_chunk(w.gpu_tokens, w.Hq, w.Hkv, w.page_size)
    max_chunks = max(-(-e // chunk) - b // chunk for b, e in zip(w.tok_begin, w.tok_end))
    desc = pkg.attn_desc(batch=w.B, num_q_heads=w.Hq, num_kv_heads=w.Hkv, head_dim=w.D, dtype=torch.float16,
                         page_size=w.page_size, num_pages=k_pool.shape[0], page_stride=k_pool.stride(0),
                         head_stride=k_pool.stride(1), tok_stride=k_pool.stride(2), block_table=block_table,
                         max_pages=block_table.shape[1], chunk_tokens=chunk, num_chunks=max_chunks)
    ws = torch.empty(pkg.hg_attn_workspace_bytes(desc, 2), dtype=torch.uint8, device=DEV)
    out = torch.empty(w.B, w.Hq, w.D, device=DEV)
    lse = torch.empty(w.B, w.Hq, device=DEV)
    i32 = lambda x: torch.tensor(x, dtype=torch.int32, device=DEV)
    pkg.hg_attn_decode(w.q(DEV), k_pool, v_pool, i32(w.seq_lens), i32(w.tok_begin), i32(w.tok_end),
                       ref.host_partials_device(DEV), out, lse, ws, desc)
    torch.cuda.synchronize()
    check_output(out, lse, ref.out, ref.lse, "readme")


@pytest.mark.parametrize("rows,slots", [(8, 65), (24, 700), (48, 300), (64, 548), (100, 131), (128, 700), (200, 300), (320, 40), (512, 70)])
def test_merge_launch_shapes_against_the_oracle(rows, slots):
    """hg_attn_merge alone on synthetic partials, over the launch shapes it chooses between (clusters of 8, 4 and 2 CTAs,
    one CTA of 8 or of 32 warps per row), with and without clusters: against the oracle's MERGE."""
    from oracle import hg_oracle as O
    D, B = 128, 1
    g = torch.Generator(device=DEV).manual_seed(rows * 1000 + slots)
    o = torch.randn(B, rows, slots, D, device=DEV, generator=g)
    m = torch.randn(B, rows, slots, device=DEV, generator=g) * 3.0
    l = torch.rand(B, rows, slots, device=DEV, generator=g) * 50.0 + 1.0
    m[:, :, slots // 2:] = float("-inf")                                     # trailing empty slots ...
    m[:, ::3, : slots // 4] = float("-inf"); m[:, 1, :] = float("-inf")      # ... holes, and a row with nothing at all
    host = (torch.randn(B, rows, 1, D, device=DEV, generator=g), torch.randn(B, rows, 1, device=DEV, generator=g) + 2.0,
            torch.rand(B, rows, 1, device=DEV, generator=g) + 1.0)
    host[1][:, 1] = float("-inf")
    outs = []
    for tune in (0, hg.HG_TUNE_NO_MERGE_CLUSTER):
        desc = pkg.attn_desc(batch=B, num_q_heads=rows, num_kv_heads=rows, head_dim=D, dtype=torch.float16, page_size=16, num_pages=1,
                             page_stride=16 * rows * D, head_stride=16 * D, tok_stride=D, block_table=None, max_pages=1,
                             chunk_tokens=64, num_chunks=slots, tune=tune)
        out = torch.full((B, rows, D), 9.0, device=DEV); lse = torch.full((B, rows), 9.0, device=DEV)
        pkg.hg_attn_merge([(o, m, l), host], out, lse, desc)
        torch.cuda.synchronize()
        outs.append((out, lse))
    mm = torch.cat([m, host[1]], dim=2).double().cpu().numpy(); ll = torch.cat([l, host[2]], dim=2).double().cpu().numpy()
    oo = torch.cat([o, host[0]], dim=2).double().cpu().numpy()
    ref_out, ref_lse = O.merge_batch(mm, ll, oo)
    for out, lse in outs:
        got, gl = out.double().cpu().numpy(), lse.double().cpu().numpy()
        assert np.all(got[0, 1] == 0.0) and gl[0, 1] == -np.inf                 # the empty row
        keep = np.isfinite(ref_lse)
        assert np.abs(got[keep] - ref_out[keep]).max() <= 1e-4 and np.abs(gl[keep] - ref_lse[keep]).max() <= 1e-4

"""The paper's literal CPU -> GPU hand-off on the GPU: the host sends logits of its (selected) tokens and
their V rows, hg_attn_partial_from_logits turns them into partials, hg_attn_merge combines them with the
partials of the GPU-resident slice.  Checked against the oracle: chunk partials one by one, and the merged
result against monolithic attention over exactly the tokens that took part."""
import numpy as np
import pytest
import torch

import paper_2604_18529_b200 as pkg
from oracle import hg_oracle as O
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import LSE_ABS, OUT_MAX_ABS, OUT_REL_L2, bits, check_partials

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


# both kernels of the hand-off: warp-level MMAs, and tcgen05.mma with the accumulator in tensor memory
KERNELS = [pytest.param(pkg.binding.HG_LOGITS_TUNE_WARP_MMA, id="warp_mma"), pytest.param(pkg.binding.HG_LOGITS_TUNE_TCGEN05, id="tcgen05")]


def handoff_case(w, keep, chunk, seed=0):
    """keep: fraction of the host slice the host selects (top logits of the group's first head, per KV head)."""
    rng = np.random.default_rng(seed)
    q, K, V = bits(w.q()), bits(w.kv_logical("k")), bits(w.kv_logical("v"))
    G = w.G
    n_host = [tb for tb in w.tok_begin]                           # the host holds [0, tok_begin)
    Ksel = max(1, max(int(np.ceil(keep * n)) for n in n_host))
    Kpad = Ksel + 5                                               # a few slots that are never used
    logits = np.full((w.B, w.Hq, Kpad), -np.inf)
    vrows = np.zeros((w.B, w.Hkv, Kpad, w.D), dtype=np.uint16)
    vrows[:] = 0x7E00                                             # NaN patterns in unused slots must not matter
    n_sel = np.zeros(w.B, dtype=np.int32)
    chosen = {}
    for b in range(w.B):
        k = int(np.ceil(keep * n_host[b])) if n_host[b] else 0
        n_sel[b] = k
        for g in range(w.Hkv):
            Kr, Vr = np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g])
            if k == 0:
                chosen[(b, g)] = np.zeros(0, dtype=np.int64)
                continue
            s0 = O.logits(q[b, g * G], Kr, w.dtype, t0=0, n=n_host[b])
            idx = np.sort(np.argsort(-s0)[:k]) if keep < 1.0 else np.arange(n_host[b])
            idx = rng.permutation(idx)                            # slot order is arbitrary
            chosen[(b, g)] = idx
            vrows[b, g, :k] = Vr[idx]
            for hh in range(G):
                logits[b, g * G + hh, :k] = O.logits(q[b, g * G + hh], Kr, w.dtype, idx=idx)
    if w.B > 1 and n_sel[1] > 3:                                  # head 0 of sequence 1 drops some of its slots
        logits[1, 0, 1:n_sel[1]:3] = -np.inf
    return q, K, V, logits, vrows, n_sel, chosen, Kpad


@pytest.mark.parametrize("G,D,dtype", [(1, 128, "f16"), (4, 128, "f16"), (8, 64, "bf16"), (12, 128, "bf16")])
@pytest.mark.parametrize("keep,chunk", [(1.0, 256), (0.25, 64), (0.05, 32)])
@pytest.mark.parametrize("kernel", KERNELS)
def test_handoff_partials_and_merged_result(G, D, dtype, keep, chunk, kernel):
    w = W.AttnWorkload("handoff", 3, 2 * G, 2, D, dtype, [900, 400, 130], [500, 333, 0], [900, 400, 130],
                       page_size=16, chunk_tokens=128, seed=41 + G)
    q, K, V, logits, vrows, n_sel, chosen, Kpad = handoff_case(w, keep, chunk)
    NCs = -(-Kpad // chunk)
    desc = pkg.logits_desc(batch=w.B, num_q_heads=w.Hq, num_kv_heads=w.Hkv, head_dim=D, dtype=dtype,
                           max_selected=Kpad, chunk_tokens=chunk, num_chunks=NCs, tune=kernel)
    lg = torch.from_numpy(logits).float().to(DEV)
    vr = torch.from_numpy(vrows.view(np.int16)).to(DEV)
    ns = torch.from_numpy(n_sel).to(DEV)
    ho = torch.full((w.B, w.Hq, NCs, D), 5.0, device=DEV); hm = torch.full((w.B, w.Hq, NCs), 5.0, device=DEV)
    hl = torch.full((w.B, w.Hq, NCs), 5.0, device=DEV)
    pkg.hg_attn_partial_from_logits(lg, vr, ns, ho, hm, hl, desc)

    # chunk partials against the oracle, fed with the fp32 logits the GPU saw
    lg32 = lg.double().cpu().numpy()
    rm = np.full((w.B, w.Hq, NCs), -np.inf); rl = np.zeros((w.B, w.Hq, NCs)); ro = np.zeros((w.B, w.Hq, NCs, D))
    for b in range(w.B):
        for h in range(w.Hq):
            for c in range(NCs):
                a, e = c * chunk, min((c + 1) * chunk, int(n_sel[b]))
                if e > a:
                    rm[b, h, c], rl[b, h, c], ro[b, h, c] = O.partial_from_logits(lg32[b, h, a:e], vrows[b, h // w.G, a:e], dtype)
    torch.cuda.synchronize()
    check_partials(ho.reshape(-1, D), hm.reshape(-1), hl.reshape(-1), rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, D))

    # merged with the GPU slice's partials: monolithic attention over the GPU slice plus the selected host tokens
    prob = DeviceProblem(w, DEV)
    prob.partial()
    prob.merge([(ho, hm, hl)])
    torch.cuda.synchronize()
    out, lse = prob.out.double().cpu().numpy(), prob.lse.double().cpu().numpy()
    ref_out = np.zeros_like(out); ref_lse = np.zeros_like(lse)
    for b in range(w.B):
        for h in range(w.Hq):
            g = h // w.G
            host = chosen[(b, g)]
            if b == 1 and h == 0 and len(host) > 3:
                drop = np.zeros(len(host), dtype=bool); drop[1::3] = True
                host = host[~drop]
            tokens = np.concatenate([host, np.arange(w.tok_begin[b], w.tok_end[b])]).astype(np.int64)
            Kr, Vr = np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g])
            ref_out[b, h], ref_lse[b, h] = O.full(q[b, h], Kr, Vr, dtype, idx=tokens)
            if keep == 1.0 and not (b == 1 and h == 0):
                lo, ll = O.literal(q[b, h], Kr, Vr, dtype, np.sort(host), np.arange(w.tok_begin[b], w.tok_end[b]))
                assert np.abs(lo - ref_out[b, h]).max() < 1e-12 and abs(ll - ref_lse[b, h]) < 1e-12
    assert np.abs(out - ref_out).max() <= OUT_MAX_ABS
    assert np.linalg.norm(out - ref_out) / np.linalg.norm(ref_out) <= OUT_REL_L2
    assert np.abs(lse - ref_lse).max() <= LSE_ABS


@pytest.mark.parametrize("G,D,dtype,K,chunk", [(1, 64, "f16", 77, 96), (16, 64, "bf16", 333, 96), (3, 128, "f16", 1025, 1024),
                                               (8, 128, "bf16", 2049, 160), (5, 128, "f16", 64, 64)])
@pytest.mark.parametrize("kernel", KERNELS)
def test_handoff_odd_sizes(G, D, dtype, K, chunk, kernel):
    """Row lengths that are not a multiple of anything (logit rows at odd offsets take the scalar load path, V tiles
    straddle the end of a chunk and of the whole array), chunk sizes that are not a multiple of the 64-row tile, groups
    that fill one and a half or two head blocks, empty sequences and sequences that use every slot."""
    rng = np.random.default_rng(K + G)
    B, Hkv = 3, 2
    Hq = Hkv * G
    n_sel = np.array([K, 0, max(1, K // 3)], dtype=np.int32)
    logits = (rng.standard_normal((B, Hq, K)) * 3.0).astype(np.float32)
    logits[0, 0, ::5] = -np.inf                                     # a head that drops slots
    v = (rng.standard_normal((B, Hkv, K, D)) * 2.0).astype(np.float32)
    vt = torch.from_numpy(v).to(torch.float16 if dtype == "f16" else torch.bfloat16)
    vbits = bits(vt)
    for b in range(B):                                              # rows past n_sel: NaN patterns that must never matter
        vbits[b, :, n_sel[b]:] = 0x7E00 if dtype == "f16" else 0x7FC0
    NCs = -(-K // chunk)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    desc = pkg.logits_desc(batch=B, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, dtype=dtype, max_selected=K,
                           chunk_tokens=chunk, num_chunks=NCs, status=status, tune=kernel)
    lg = torch.from_numpy(logits).to(DEV)
    vr = torch.from_numpy(vbits.view(np.int16)).to(DEV)
    ho = torch.full((B, Hq, NCs, D), 5.0, device=DEV); hm = torch.full((B, Hq, NCs), 5.0, device=DEV); hl = torch.full_like(hm, 5.0)
    pkg.hg_attn_partial_from_logits(lg, vr, torch.from_numpy(n_sel).to(DEV), ho, hm, hl, desc)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    rm = np.full((B, Hq, NCs), -np.inf); rl = np.zeros((B, Hq, NCs)); ro = np.zeros((B, Hq, NCs, D))
    for b in range(B):
        for h in range(Hq):
            for c in range(NCs):
                a, e = c * chunk, min((c + 1) * chunk, int(n_sel[b]))
                if e > a:
                    rm[b, h, c], rl[b, h, c], ro[b, h, c] = O.partial_from_logits(logits[b, h, a:e].astype(np.float64), vbits[b, h // G, a:e], dtype)
    check_partials(ho.reshape(-1, D), hm.reshape(-1), hl.reshape(-1), rm.reshape(-1), rl.reshape(-1), ro.reshape(-1, D))


def test_handoff_rejects_bad_descriptions():
    from paper_2604_18529_b200 import binding as hg
    t = torch.zeros(8, device=DEV)
    ti = torch.zeros(8, dtype=torch.int32, device=DEV)
    for bad in (dict(chunk_tokens=48), dict(chunk_tokens=2048), dict(num_chunks=1, max_selected=4096), dict(head_dim=96)):
        kw = dict(batch=1, num_q_heads=2, num_kv_heads=1, head_dim=128, dtype="f16", max_selected=64, chunk_tokens=64)
        kw.update(bad)
        with pytest.raises(hg.HgError):
            pkg.hg_attn_partial_from_logits(t, t.half(), ti, t, t, t, pkg.logits_desc(**kw))


# ---- the whole CPU stage with the library's own host functions ---------------------------------------------------

@pytest.mark.parametrize("strategy", ["post_qk", "pre_qk"])
@pytest.mark.parametrize("G", [1, 4])
def test_cpu_stage_feeds_the_gpu_stage(strategy, G):
    """Post-QK^T: host logits for every offloaded token, top-K per KV head (score = best head of the group),
    Pre-QK^T: sinks + recent window chosen before any logit is computed; then logits of the chosen tokens and
    their V rows cross to the GPU, which merges them with its own slice.  Equal to monolithic attention over
    exactly those tokens."""
    from paper_2604_18529_b200 import host as H
    w = W.AttnWorkload("stage", 2, 2 * G, 2, 128, "f16", [1500, 700], [1100, 420], [1500, 700], page_size=16,
                       chunk_tokens=128, seed=60 + G, outlier_frac=0.02)
    q_t, K_t, V_t = w.q(), w.kv_logical("k"), w.kv_logical("v")
    n_host = torch.tensor(w.tok_begin, dtype=torch.int32)
    Ksel = 96
    if strategy == "post_qk":
        all_logits = torch.empty(w.B, w.Hq, int(n_host.max()))
        H.hg_host_logits(q_t, K_t, None, n_host, all_logits, H.host_desc(K_t, w.Hq, int(n_host.max())))
        score = all_logits.view(w.B, w.Hkv, G, -1).max(dim=2).values.reshape(w.B * w.Hkv, -1).contiguous()
        idx, n_out = H.hg_host_select_topk(score, n_host.repeat_interleave(w.Hkv), Ksel)
        idx = idx.view(w.B, w.Hkv, Ksel)
        n_sel = n_out.view(w.B, w.Hkv)[:, 0].contiguous()
    else:
        idx = torch.full((w.B, w.Hkv, Ksel), -1, dtype=torch.int32)
        n_sel = torch.zeros(w.B, dtype=torch.int32)
        for b in range(w.B):
            sel = H.hg_host_select_positions(int(n_host[b]), 4, 64, Ksel)
            idx[b, :, : len(sel)] = sel
            n_sel[b] = len(sel)
    desc = H.host_desc(K_t, w.Hq, Ksel)
    logits = torch.empty(w.B, w.Hq, Ksel)
    H.hg_host_logits(q_t, K_t, idx, n_sel, logits, desc)
    vsel = torch.empty(w.B, w.Hkv, Ksel, w.D, dtype=torch.float16)
    H.hg_host_gather_rows(V_t, idx, n_sel, vsel, desc)

    ld = pkg.logits_desc(batch=w.B, num_q_heads=w.Hq, num_kv_heads=w.Hkv, head_dim=w.D, dtype=w.dtype, max_selected=Ksel,
                         chunk_tokens=32)
    NCs = ld.num_chunks
    ho = torch.empty(w.B, w.Hq, NCs, w.D, device=DEV); hm = torch.empty(w.B, w.Hq, NCs, device=DEV); hl = torch.empty_like(hm)
    pkg.hg_attn_partial_from_logits(logits.to(DEV), vsel.to(DEV), n_sel.to(DEV), ho, hm, hl, ld)
    prob = DeviceProblem(w, DEV)
    prob.partial()
    prob.merge([(ho, hm, hl)])
    torch.cuda.synchronize()

    q, K, V = bits(q_t), bits(K_t), bits(V_t)
    out, lse = prob.out.double().cpu().numpy(), prob.lse.double().cpu().numpy()
    ref_out = np.zeros_like(out); ref_lse = np.zeros_like(lse)
    for b in range(w.B):
        for h in range(w.Hq):
            g = h // G
            host = idx[b, g, : int(n_sel[b])].numpy().astype(np.int64)
            assert len(set(host.tolist())) == len(host) and (host < w.tok_begin[b]).all()
            tokens = np.concatenate([host, np.arange(w.tok_begin[b], w.tok_end[b])])
            ref_out[b, h], ref_lse[b, h] = O.full(q[b, h], np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g]),
                                                  w.dtype, idx=tokens)
    assert np.abs(out - ref_out).max() <= OUT_MAX_ABS
    assert np.linalg.norm(out - ref_out) / np.linalg.norm(ref_out) <= OUT_REL_L2
    assert np.abs(lse - ref_lse).max() <= LSE_ABS


@pytest.mark.parametrize("B,Hq,Hkv,K,chunk", [(8, 40, 40, 8192, 256), (1, 64, 8, 262144, 256), (8, 40, 40, 8192, 512), (1, 64, 8, 262144, 512)])
def test_handoff_at_the_sizes_and_launch_configurations_the_bench_times(B, Hq, Hkv, K, chunk):
    """The four hand-off measurements of bench.py (0.6 - 0.7 GB each, the library's own choice of kernel: warp-level MMAs
    at 256-slot chunks, tcgen05 at 512): sampled (sequence, head, chunk) partials against the oracle, and properties
    that hold for every partial."""
    D, G = 128, Hq // Hkv
    gen = torch.Generator(device=DEV).manual_seed(11)
    logits = torch.randn(B, Hq, K, device=DEV, generator=gen)
    vrows = torch.randn(B, Hkv, K, D, device=DEV, generator=gen).half()
    n_sel = torch.full((B,), K, dtype=torch.int32, device=DEV)
    n_sel[-1] = K - 37                                             # a ragged last chunk in the last sequence
    ld = pkg.logits_desc(batch=B, num_q_heads=Hq, num_kv_heads=Hkv, head_dim=D, dtype="f16", max_selected=K, chunk_tokens=chunk)
    NC = ld.num_chunks
    o = torch.full((B, Hq, NC, D), 7.0, device=DEV); m = torch.full((B, Hq, NC), 7.0, device=DEV); l = torch.full((B, Hq, NC), 7.0, device=DEV)
    pkg.hg_attn_partial_from_logits(logits, vrows, n_sel, o, m, l, ld)
    torch.cuda.synchronize()
    # every partial: the maximum is the chunk's largest logit, 1 <= l <= slots in use, nothing left unwritten
    ref_m = logits.view(B, Hq, NC, chunk).amax(dim=3)
    ref_m[-1, :, -1] = logits[-1, :, (NC - 1) * chunk:K - 37].amax(dim=1)
    assert torch.equal(m, ref_m)
    assert bool((l >= 1.0).all()) and bool((l <= chunk).all()) and bool(torch.isfinite(o).all())
    # sampled partials against the oracle (first and last chunk of the ragged sequence among them)
    rng = np.random.default_rng(5)
    picks = [(B - 1, Hq - 1, NC - 1), (B - 1, 0, NC - 1), (0, 0, 0)] + [(int(rng.integers(B)), int(rng.integers(Hq)), int(rng.integers(NC))) for _ in range(45)]
    got_o, got_m, got_l, rm, rl, ro = [], [], [], [], [], []
    for b, h, c in picks:
        a, e = c * chunk, min((c + 1) * chunk, int(n_sel[b]))
        lg = logits[b, h, a:e].double().cpu().numpy()
        vr = vrows[b, h // G, a:e].contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
        mm, ll, oo = O.partial_from_logits(lg, vr, "f16")
        rm.append(mm); rl.append(ll); ro.append(oo)
        got_o.append(o[b, h, c]); got_m.append(m[b, h, c]); got_l.append(l[b, h, c])
    check_partials(torch.stack(got_o), torch.stack(got_m), torch.stack(got_l), np.array(rm), np.array(rl), np.stack(ro))

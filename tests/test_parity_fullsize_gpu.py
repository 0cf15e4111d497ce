"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every (sequence, head) row of the four large configurations is compared with the fp64 oracle: the chunk
partials (m, m + ln l, o / l), the merged output and the LSE, with the whole-tensor relative L2 error as the
gate and the worst row reported.  The logical K and V rows of a few KV heads at a time are produced on the
GPU by the seeded generator, handed to the oracle as bit patterns, and the oracle's rows run on all host
cores; a handful of rows are also computed as monolithic attention (FULL) to confirm, at full size, that the
oracle's merged reference is the unsplit result.  Properties that hold at any size close the test."""
import time

import numpy as np
import pytest
import torch

from oracle import hg_oracle as O
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import LSE_ABS, OUT_MAX_ABS, OUT_REL_L2, bits, check_output, check_partials

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def sample_rows(w):
    rows = {(0, 0), (w.B - 1, w.Hq - 1), (w.B // 2, w.Hq // 2 + 1 if w.Hq > 2 else 0)}
    if w.name == "ragged":      # the shortest and the longest GPU slice
        n = [e - b for b, e in zip(w.tok_begin, w.tok_end)]
        rows |= {(int(np.argmin(n)), 3), (int(np.argmax(n)), w.Hq - 2)}
    return sorted(rows)


def oracle_every_row(w, NC):
    """Chunk partials of the GPU slice, the host-held slice's partial and the merged reference for every row."""
    B, Hq, Hkv, G, D, C = w.B, w.Hq, w.Hkv, w.G, w.D, w.chunk_tokens
    ref_m = np.empty((B, Hq, NC)); ref_l = np.empty((B, Hq, NC)); ref_o = np.empty((B, Hq, NC, D))
    host_m = np.empty((B, Hq, 1)); host_l = np.empty((B, Hq, 1)); host_o = np.empty((B, Hq, 1, D))
    full_rows = {}
    q_all = bits(w.q())
    sampled = set(sample_rows(w))
    per_call = max(1, -(-O.host_threads() // G))           # KV heads per oracle call: a row per host core at least
    for b in range(B):
        L, tb, te = w.seq_lens[b], w.tok_begin[b], w.tok_end[b]
        assert tb > 0 and te == L                           # suffix slices: the host holds [0, tb)
        for g0 in range(0, Hkv, per_call):
            gs = list(range(g0, min(Hkv, g0 + per_call)))
            K = bits(torch.stack([w.kv_rows("k", b, g, 0, L, DEV) for g in gs], dim=1))[None]     # [1][L][heads][D]
            V = bits(torch.stack([w.kv_rows("v", b, g, 0, L, DEV) for g in gs], dim=1))[None]
            h0, h1 = gs[0] * G, (gs[-1] + 1) * G
            q = q_all[b:b + 1, h0:h1]
            m, l, o = O.chunked_partials(q, K, V, w.dtype, [tb], [te], C, NC)
            ref_m[b, h0:h1], ref_l[b, h0:h1], ref_o[b, h0:h1] = m[0], l[0], o[0]
            m, l, o = O.chunked_partials(q, K, V, w.dtype, [0], [tb], 0, 1)
            host_m[b, h0:h1], host_l[b, h0:h1], host_o[b, h0:h1] = m[0], l[0], o[0]
            for (bb, h) in sampled:
                if bb == b and h0 <= h < h1:
                    j = (h - h0) // G
                    full_rows[(b, h)] = O.full(q_all[b, h], np.ascontiguousarray(K[0, :, j]), np.ascontiguousarray(V[0, :, j]), w.dtype)
            del K, V
    out, lse = O.merge_batch(np.concatenate([host_m, ref_m], axis=2), np.concatenate([host_l, ref_l], axis=2),
                             np.concatenate([host_o, ref_o], axis=2))
    # the exactness claim at full size, inside the oracle: merged partials = monolithic attention
    for (b, h), (fo, fl) in full_rows.items():
        assert np.abs(out[b, h] - fo).max() < 1e-11 and abs(lse[b, h] - fl) < 1e-10, (b, h)
    assert len(full_rows) == len(sampled)
    return (ref_m, ref_l, ref_o), (host_m, host_l, host_o), (out, lse)


@pytest.mark.parametrize("name", ["opt13b", "opt30b", "llama70b", "ragged"])
def test_full_size_every_row(name):
    w = W.make_workload(name)
    prob = DeviceProblem(w, DEV)
    C, NC, D = w.chunk_tokens, prob.NC, w.D
    t0 = time.time()
    (ref_m, ref_l, ref_o), (host_m, host_l, host_o), (ref_out, ref_lse) = oracle_every_row(w, NC)
    t_oracle = time.time() - t0

    f32 = lambda a: torch.from_numpy(a).float().to(DEV)
    prob.step([(f32(host_o), f32(host_m), f32(host_l))])
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK

    check_partials(prob.o_part, prob.m_part, prob.l_part, ref_m, ref_l, ref_o, name)
    max_abs, rel, lerr = check_output(prob.out, prob.lse, ref_out, ref_lse, name)        # whole-tensor gates
    out, lse = prob.out.cpu().double().numpy(), prob.lse.cpu().double().numpy()
    row_abs = np.abs(out - ref_out).max(axis=2)
    row_rel = np.linalg.norm(out - ref_out, axis=2) / np.linalg.norm(ref_out, axis=2)
    row_lse = np.abs(lse - ref_lse)
    assert row_abs.max() <= OUT_MAX_ABS and row_rel.max() <= OUT_REL_L2 and row_lse.max() <= LSE_ABS   # and the worst row
    wb, wh = np.unravel_index(np.argmax(row_rel), row_rel.shape)
    print(f"{name}: rows = {w.B * w.Hq} of {w.B * w.Hq}, whole tensor max_abs {max_abs:.2e} rel_l2 {rel:.2e} lse {lerr:.2e}; "
          f"worst row (b={wb}, h={wh}) max_abs {row_abs.max():.2e} rel_l2 {row_rel.max():.2e} lse {row_lse.max():.2e}; "
          f"oracle {t_oracle:.1f} s on {O.host_threads()} cores")

    # properties that hold for every row at any size
    m_part, l_part = prob.m_part.cpu().double().numpy(), prob.l_part.cpu().double().numpy()
    assert not np.isnan(out).any() and not np.isnan(lse).any() and np.isfinite(lse).all()
    live = np.isfinite(m_part)
    for b in range(w.B):
        n_b = w.chunk_grid(b)[1]
        assert live[b, :, :n_b].all() and not live[b, :, n_b:].any()
    assert (l_part[live] >= 1.0 - 1e-6).all() and (l_part[live] <= C * (1 + 1e-5)).all()
    assert (l_part[~live] == 0).all()
    vmax = 4.4 * w.sigma_kv * (w.outlier_scale if w.outlier_frac > 0 else 1.0)     # the generator's largest |value|
    assert np.abs(out).max() <= vmax

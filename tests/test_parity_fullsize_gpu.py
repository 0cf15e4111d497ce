"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The whole-tensor oracle would take minutes here, so a few (sequence, head) rows are checked one by
one against the oracle - chunk partials, merged output and LSE - and every row is checked against
properties that hold at any size (no NaN, exp-sums within [1, chunk length], output inside the
range of V)."""
import numpy as np
import pytest
import torch

from oracle import hg_oracle as O
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import workload as W
from paper_2604_18529_b200.problem import DeviceProblem
from parity_util import LSE_ABS, OUT_MAX_ABS, OUT_REL_L2, bits

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def sample_rows(w):
    rows = {(0, 0), (w.B - 1, w.Hq - 1), (w.B // 2, w.Hq // 2 + 1 if w.Hq > 2 else 0)}
    if w.name == "ragged":      # the shortest and the longest GPU slice
        n = [e - b for b, e in zip(w.tok_begin, w.tok_end)]
        rows |= {(int(np.argmin(n)), 3), (int(np.argmax(n)), w.Hq - 2)}
    return sorted(rows)


@pytest.mark.parametrize("name", ["opt13b", "opt30b", "llama70b", "ragged"])
def test_full_size_sampled_rows(name):
    w = W.make_workload(name)
    prob = DeviceProblem(w, DEV)
    rows = sample_rows(w)
    q_all = w.q()
    C, NC, D = w.chunk_tokens, prob.NC, w.D

    host_o = torch.zeros(w.B, w.Hq, 1, D)
    host_m = torch.full((w.B, w.Hq, 1), float("-inf"))
    host_l = torch.zeros(w.B, w.Hq, 1)
    refs = {}
    for b, h in rows:
        g, L, tb, te = h // w.G, w.seq_lens[b], w.tok_begin[b], w.tok_end[b]
        K = bits(w.kv_rows("k", b, g, 0, L, DEV))
        V = bits(w.kv_rows("v", b, g, 0, L, DEV))
        q = bits(q_all[b, h])
        assert tb > 0 and te == L                                   # suffix slices: the host holds [0, tb)
        hm, hl, ho = O.partial(q, K, V, w.dtype, t0=0, n=tb)
        host_o[b, h, 0] = torch.from_numpy(ho).float(); host_m[b, h, 0] = hm; host_l[b, h, 0] = hl
        # the GPU slice chunk by chunk on the absolute chunk grid, and monolithic attention over everything
        first = tb // C
        chunks = []
        for c in range(NC):
            a, e = max((first + c) * C, tb), min((first + c + 1) * C, te)
            chunks.append(O.partial(q, K, V, w.dtype, t0=a, n=max(0, e - a)))
        refs[(b, h)] = (chunks, O.full(q, K, V, w.dtype))
        # the exactness claim, at full size, inside the oracle itself
        mo, ml = O.merge([hm] + [c[0] for c in chunks], [hl] + [c[1] for c in chunks], [ho] + [c[2] for c in chunks])
        assert np.abs(mo - refs[(b, h)][1][0]).max() < 1e-11 and abs(ml - refs[(b, h)][1][1]) < 1e-10

    prob.step([(host_o.to(DEV), host_m.to(DEV), host_l.to(DEV))])
    torch.cuda.synchronize()
    assert int(prob.status.item()) == hg.HG_DEV_OK

    o_part, m_part, l_part = prob.o_part.cpu().double().numpy(), prob.m_part.cpu().double().numpy(), prob.l_part.cpu().double().numpy()
    out, lse = prob.out.cpu().double().numpy(), prob.lse.cpu().double().numpy()
    worst = [0.0, 0.0, 0.0]
    for (b, h), (chunks, (ref_out, ref_lse)) in refs.items():
        for c, (rm, rl, ro) in enumerate(chunks):
            if rm == -np.inf:
                assert m_part[b, h, c] == -np.inf and l_part[b, h, c] == 0 and not o_part[b, h, c].any()
                continue
            assert abs(m_part[b, h, c] - rm) <= LSE_ABS
            assert abs(m_part[b, h, c] + np.log(l_part[b, h, c]) - (rm + np.log(rl))) <= LSE_ABS
            assert np.abs(o_part[b, h, c] / l_part[b, h, c] - ro / rl).max() <= OUT_MAX_ABS
        err = np.abs(out[b, h] - ref_out).max()
        rel = np.linalg.norm(out[b, h] - ref_out) / np.linalg.norm(ref_out)
        lerr = abs(lse[b, h] - ref_lse)
        worst = [max(worst[0], err), max(worst[1], rel), max(worst[2], lerr)]
        assert err <= OUT_MAX_ABS and rel <= OUT_REL_L2 and lerr <= LSE_ABS, (name, b, h, err, rel, lerr)
    print(f"{name}: rows {len(refs)} max_abs {worst[0]:.2e} rel_l2 {worst[1]:.2e} lse {worst[2]:.2e}")

    # properties that hold for every row at any size
    assert not np.isnan(out).any() and not np.isnan(lse).any() and np.isfinite(lse).all()
    live = np.isfinite(m_part)
    for b in range(w.B):
        n_b = w.chunk_grid(b)[1]
        assert live[b, :, :n_b].all() and not live[b, :, n_b:].any()
    assert (l_part[live] >= 1.0 - 1e-6).all() and (l_part[live] <= C * (1 + 1e-5)).all()
    assert (l_part[~live] == 0).all()
    vmax = 4.4 * w.sigma_kv * (w.outlier_scale if w.outlier_frac > 0 else 1.0)     # the generator's largest |value|
    assert np.abs(out).max() <= vmax

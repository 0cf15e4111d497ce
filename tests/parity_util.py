"""Helpers for the GPU-vs-oracle parity tests: oracle references for a workload and error measures."""

import numpy as np
import torch

from oracle import hg_oracle as O

# tolerances of the GPU path against the fp64 oracle (fp16/bf16 KV, fp32 accumulation)
OUT_MAX_ABS = 2e-3
OUT_REL_L2 = 1e-3
LSE_ABS = 1e-4


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


class OracleRef:
    """Everything the oracle says about a (small) workload, from its logical cache."""

    def __init__(self, w):
        self.w = w
        self.q = bits(w.q())
        self.K = bits(w.kv_logical("k"))
        self.V = bits(w.kv_logical("v"))
        zeros = [0] * w.B
        # monolithic attention over the whole sequence
        self.out, self.lse = O.full_batch(self.q, self.K, self.V, w.dtype, zeros, w.seq_lens)
        # host-held slice: tokens before and after the GPU slice, one partial each
        self.host = [O.chunked_partials(self.q, self.K, self.V, w.dtype, lo, hi, 0, 1)
                     for lo, hi in ((zeros, w.tok_begin), (w.tok_end, w.seq_lens))]

    def chunk_partials(self, chunk, NC):
        return O.chunked_partials(self.q, self.K, self.V, self.w.dtype, self.w.tok_begin, self.w.tok_end, chunk, NC)

    def host_partials_device(self, device):
        return [tuple(torch.from_numpy(x).float().to(device) for x in (o, m, l)) for (m, l, o) in self.host]


def check_output(out, lse, ref_out, ref_lse, what=""):
    out = out.double().cpu().numpy(); lse = lse.double().cpu().numpy()
    assert not np.isnan(out).any() and not np.isnan(lse).any(), what
    max_abs = np.abs(out - ref_out).max()
    rel = np.linalg.norm(out - ref_out) / max(np.linalg.norm(ref_out), 1e-300)
    finite = np.isfinite(ref_lse)
    assert np.array_equal(np.isfinite(lse), finite), what
    lerr = np.abs(lse[finite] - ref_lse[finite]).max() if finite.any() else 0.0
    assert np.array_equal(lse[~finite], ref_lse[~finite]), what
    assert max_abs <= OUT_MAX_ABS, f"{what}: out max abs {max_abs:.3e}"
    assert rel <= OUT_REL_L2, f"{what}: out rel L2 {rel:.3e}"
    assert lerr <= LSE_ABS, f"{what}: lse abs {lerr:.3e}"
    return max_abs, rel, lerr


def check_partials(o, m, l, ref_m, ref_l, ref_o, what=""):
    """Chunk partials against the oracle: the exact chunk maximum, and the representation-free
    quantities m + ln l and o / l."""
    o = o.double().cpu().numpy(); m = m.double().cpu().numpy(); l = l.double().cpu().numpy()
    empty = np.isinf(ref_m)
    assert np.array_equal(np.isinf(m) & (m < 0), empty), what
    assert (l[empty] == 0).all() and (o[empty] == 0).all(), what
    live = ~empty
    if not live.any():
        return
    assert np.abs(m[live] - ref_m[live]).max() <= LSE_ABS, f"{what}: chunk max"
    assert np.abs((m[live] + np.log(l[live])) - (ref_m[live] + np.log(ref_l[live]))).max() <= LSE_ABS, f"{what}: chunk lse"
    a = o[live] / l[live][:, None]
    r = ref_o[live] / ref_l[live][:, None]
    assert np.abs(a - r).max() <= OUT_MAX_ABS, f"{what}: chunk o/l max abs {np.abs(a - r).max():.3e}"
    assert np.linalg.norm(a - r) / max(np.linalg.norm(r), 1e-300) <= OUT_REL_L2, f"{what}: chunk o/l rel L2"

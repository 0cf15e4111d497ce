"""Seeded synthetic decode-attention workloads (inputs only; no attention arithmetic lives here).

Every value is a pure function of (seed, tensor id, logical coordinates), so the same
element can be produced on the CPU for the fp64 oracle and on the GPU for the kernels
without either side seeing the other's data:

    value(b, t, g, d) = round16( sigma * outlier(b, t) * GAUSS[ hash64(key, linear(b,t,g,d)) >> 48 ] )

* ``hash64`` is a SplitMix64-style finaliser evaluated with wrapping int64 torch ops,
  bit-identical on CPU and CUDA tensors.
* ``GAUSS`` is a 65536-entry fp32 table of standard-normal quantiles (mid-point rule),
  computed once on the CPU in fp64 and uploaded; a table lookup keeps the generator free
  of device-dependent transcendental functions.
* ``outlier(b, t)`` is 1 or ``outlier_scale``; a token is an outlier with probability
  ``outlier_frac`` (same decision for every head, applied to its K and V rows alike).

The configurations mirror the decode workloads the paper evaluates (OPT / Llama / Qwen
shaped layers at 2K-32K tokens and beyond, Section 5.1) with the GPU holding the most
recent tokens of each sequence (Section 4.2, device-side support) in a paged KV pool.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Tuple

import torch

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

TENSOR_Q, TENSOR_K, TENSOR_V, TENSOR_OUTLIER, TENSOR_PERM, TENSOR_LENS = 1, 2, 3, 4, 5, 6


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the signed value an int64 tensor holds."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_int(z: int) -> int:
    z &= _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def tensor_key(seed: int, tensor_id: int) -> int:
    return _mix_int(_mix_int(seed) + tensor_id * _GOLDEN)


def _lsr(x: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 tensors."""
    return (x >> s) & ((1 << (64 - s)) - 1)


def hash64(key: int, idx: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output for counter ``idx`` (int64 tensor) under ``key``; wraps mod 2^64."""
    z = idx * _s64(_GOLDEN) + _s64(key)
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


_GAUSS_CACHE = {}


def gauss_table(device) -> torch.Tensor:
    """fp32 standard-normal quantiles at (k + 0.5) / 65536, k = 0..65535."""
    dev = torch.device(device)
    if dev not in _GAUSS_CACHE:
        p = (torch.arange(65536, dtype=torch.float64) + 0.5) / 65536.0
        _GAUSS_CACHE[dev] = torch.special.ndtri(p).to(torch.float32).to(dev)
    return _GAUSS_CACHE[dev]


def torch_dtype(name: str) -> torch.dtype:
    return {"f16": torch.float16, "bf16": torch.bfloat16}[name]


@dataclasses.dataclass
class AttnWorkload:
    """One decode step of one layer: shapes, the per-sequence GPU slice and the paging."""

    name: str
    B: int
    Hq: int
    Hkv: int
    D: int
    dtype: str                      # "f16" | "bf16" (q, K and V share it)
    seq_lens: List[int]
    tok_begin: List[int]            # GPU-resident slice [tok_begin, tok_end) per sequence
    tok_end: List[int]
    page_size: int = 16
    layout: str = "HND"             # in-page order: "HND" [Hkv][page][D], "NHD" [page][Hkv][D]
    paged: bool = True              # False: contiguous [B][Lmax][Hkv][D], no block table
    page_order: str = "random"      # physical page order: "random" | "sequential"
    chunk_tokens: int = 512
    sigma_kv: float = 1.0
    outlier_frac: float = 0.0
    outlier_scale: float = 8.0
    seed: int = 1000

    # ---- derived geometry -------------------------------------------------
    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def max_len(self) -> int:
        return max(self.seq_lens) if self.seq_lens else 0

    @property
    def max_pages(self) -> int:
        return max(1, -(-self.max_len // self.page_size))

    @property
    def gpu_tokens(self) -> int:
        return sum(e - b for b, e in zip(self.tok_begin, self.tok_end))

    def chunk_grid(self, b: int) -> Tuple[int, int]:
        """(first absolute chunk index, number of chunks) of sequence b.

        Chunks sit on absolute multiples of ``chunk_tokens``; only the first and the last
        one are clipped by the slice.
        """
        tb, te, C = self.tok_begin[b], self.tok_end[b], self.chunk_tokens
        if te <= tb:
            return 0, 0
        first = tb // C
        return first, -(-te // C) - first

    @property
    def num_chunks(self) -> int:
        return max([self.chunk_grid(b)[1] for b in range(self.B)] + [1])

    def chunk_range(self, b: int, c: int) -> Tuple[int, int]:
        first, n = self.chunk_grid(b)
        if c >= n:
            return 0, 0
        C = self.chunk_tokens
        lo = max((first + c) * C, self.tok_begin[b])
        hi = min((first + c + 1) * C, self.tok_end[b])
        return lo, hi

    def kv_bytes(self) -> int:
        """Algorithmic K+V bytes of the GPU slice: 2 * N * d per layer (Section 3.1), 16-bit."""
        return self.gpu_tokens * 2 * self.Hkv * self.D * 2

    # ---- element generators ----------------------------------------------
    def _values(self, tensor_id: int, lin: torch.Tensor, tok_scale: Optional[torch.Tensor], sigma: float):
        h = hash64(tensor_key(self.seed, tensor_id), lin)
        x = gauss_table(lin.device)[_lsr(h, 48)]
        if sigma != 1.0:
            x = x * sigma
        if tok_scale is not None:
            x = x * tok_scale
        return x.to(torch_dtype(self.dtype))

    def q(self, device="cpu") -> torch.Tensor:
        """[B][Hq][D], N(0,1)."""
        lin = torch.arange(self.B * self.Hq * self.D, dtype=torch.int64, device=device)
        return self._values(TENSOR_Q, lin, None, 1.0).view(self.B, self.Hq, self.D)

    def _outlier_scale(self, b: torch.Tensor, t: torch.Tensor) -> Optional[torch.Tensor]:
        if self.outlier_frac <= 0.0:
            return None
        h = hash64(tensor_key(self.seed, TENSOR_OUTLIER), b * (1 << 32) + t)
        flag = _lsr(h, 40) < int(self.outlier_frac * (1 << 24))
        one = torch.ones((), dtype=torch.float32, device=t.device)
        return torch.where(flag, one * self.outlier_scale, one)

    def _lin(self, b, t, g, d):
        return ((b * (1 << 22) + t) * self.Hkv + g) * self.D + d

    def kv_rows(self, which: str, b: int, g: int, t0: int, t1: int, device="cpu") -> torch.Tensor:
        """Logical rows K[b, t0:t1, g, :] (or V): [t1 - t0][D]."""
        assert self.max_len <= (1 << 22)
        t = torch.arange(t0, t1, dtype=torch.int64, device=device).view(-1, 1)
        d = torch.arange(self.D, dtype=torch.int64, device=device).view(1, -1)
        bb = torch.full_like(t, b)
        sc = self._outlier_scale(bb, t)
        tid = TENSOR_K if which == "k" else TENSOR_V
        return self._values(tid, self._lin(bb, t, g, d), sc, self.sigma_kv)

    def kv_logical(self, which: str, device="cpu") -> torch.Tensor:
        """Whole logical cache [B][Lmax][Hkv][D]; rows at t >= seq_len hold 0. Small cases only."""
        out = torch.zeros(self.B, self.max_len, self.Hkv, self.D, dtype=torch_dtype(self.dtype), device=device)
        for b in range(self.B):
            for g in range(self.Hkv):
                out[b, : self.seq_lens[b], g] = self.kv_rows(which, b, g, 0, self.seq_lens[b], device)
        return out

    # ---- paging ------------------------------------------------------------
    def page_plan(self):
        """Which logical pages are GPU-resident and where they sit in the pool.

        Returns (slot_b, slot_page, block_table): for each physical page its sequence and
        logical page index (int64 CPU tensors), and the [B][max_pages] int32 table with -1
        for pages that hold no token of the GPU slice.
        """
        ps = self.page_size
        owners = []
        for b in range(self.B):
            tb, te = self.tok_begin[b], self.tok_end[b]
            if te > tb:
                owners += [(b, j) for j in range(tb // ps, -(-te // ps))]
        n = len(owners)
        if self.page_order == "random" and n > 1:
            gen = torch.Generator().manual_seed(tensor_key(self.seed, TENSOR_PERM) & 0x7FFFFFFF)
            perm = torch.randperm(n, generator=gen)
        else:
            perm = torch.arange(n)
        own = torch.tensor(owners, dtype=torch.int64).view(-1, 2)
        slot_b = torch.empty(max(n, 1), dtype=torch.int64)
        slot_page = torch.empty(max(n, 1), dtype=torch.int64)
        table = torch.full((self.B, self.max_pages), -1, dtype=torch.int32)
        if n:
            slot_b[perm] = own[:, 0]
            slot_page[perm] = own[:, 1]
            table[own[:, 0], own[:, 1]] = perm.to(torch.int32)
        else:
            slot_b.zero_()
            slot_page.zero_()
        return slot_b, slot_page, table

    def build_device_kv(self, device, poison_tail: bool = False):
        """K and V pools in their device layout plus the addressing the kernels need.

        Paged: pools are [num_pages][Hkv][page][D] (HND) or [num_pages][page][Hkv][D] (NHD),
        holding only pages that overlap the GPU slice. Contiguous: [B][Lmax_pad][Hkv][D]
        addressed as identity pages. ``poison_tail`` overwrites rows of resident pages at
        t >= seq_len with NaN patterns (those rows must never influence a result).
        Returns a dict with k, v, block_table (or None), num_pages, max_pages and the
        page/head/token strides in elements.
        """
        ps, D, H = self.page_size, self.D, self.Hkv
        dt = torch_dtype(self.dtype)
        if self.paged:
            slot_b, slot_page, table = self.page_plan()
            npages = slot_b.numel()
        else:
            mp = self.max_pages
            slot_b = torch.arange(self.B, dtype=torch.int64).repeat_interleave(mp)
            slot_page = torch.arange(mp, dtype=torch.int64).repeat(self.B)
            table = None
            npages = self.B * mp
        hnd = self.paged and self.layout == "HND"
        shape = (npages, H, ps, D) if hnd else (npages, ps, H, D)
        pools = {}
        seq_len_t = torch.tensor(self.seq_lens, dtype=torch.int64, device=device)
        step = max(1, (1 << 25) // (H * ps * D))
        r = torch.arange(ps, dtype=torch.int64, device=device)
        g = torch.arange(H, dtype=torch.int64, device=device)
        d = torch.arange(D, dtype=torch.int64, device=device)
        for which, tid in (("k", TENSOR_K), ("v", TENSOR_V)):
            pool = torch.empty(shape, dtype=dt, device=device)
            for p0 in range(0, npages, step):
                p1 = min(npages, p0 + step)
                sb = slot_b[p0:p1].to(device)
                t = slot_page[p0:p1].to(device).view(-1, 1) * ps + r.view(1, -1)      # [P][ps]
                bb = sb.view(-1, 1).expand_as(t)
                sc = self._outlier_scale(bb, t)
                if hnd:
                    lin = self._lin(bb[:, None, :, None], t[:, None, :, None], g.view(1, -1, 1, 1), d.view(1, 1, 1, -1))
                    scv = None if sc is None else sc[:, None, :, None]
                    live = (t < seq_len_t[sb].view(-1, 1))[:, None, :, None]
                else:
                    lin = self._lin(bb[:, :, None, None], t[:, :, None, None], g.view(1, 1, -1, 1), d.view(1, 1, 1, -1))
                    scv = None if sc is None else sc[:, :, None, None]
                    live = (t < seq_len_t[sb].view(-1, 1))[:, :, None, None]
                vals = self._values(tid, lin, scv, self.sigma_kv)
                fill = float("nan") if poison_tail else 0.0
                pool[p0:p1] = torch.where(live, vals, torch.full((), fill, dtype=dt, device=device))
            pools[which] = pool
        if hnd:
            strides = dict(page_stride=H * ps * D, head_stride=ps * D, tok_stride=D)
        else:
            strides = dict(page_stride=ps * H * D, head_stride=D, tok_stride=H * D)
        return dict(k=pools["k"], v=pools["v"],
                    block_table=None if table is None else table.to(device),
                    num_pages=npages, max_pages=self.max_pages, **strides)


# ---- the five benchmark configurations ---------------------------------------

def _suffix(seq_lens, shares):
    n = [int(math.floor(s * L)) for s, L in zip(shares, seq_lens)]
    return [L - k for L, k in zip(seq_lens, n)], list(seq_lens)


def first_sequences(w: AttnWorkload, batch: int) -> AttnWorkload:
    """The same workload restricted to its first `batch` sequences (for small profiling captures)."""
    batch = max(1, min(batch, w.B))
    return dataclasses.replace(w, name=f"{w.name}[:{batch}]", B=batch, seq_lens=w.seq_lens[:batch],
                               tok_begin=w.tok_begin[:batch], tok_end=w.tok_end[:batch])


def make_workload(name: str) -> AttnWorkload:
    if name == "tiny":
        # prefix slice on the GPU, contiguous cache
        return AttnWorkload("tiny", 1, 8, 8, 64, "f16", [2048], [0], [1024], page_size=64,
                            layout="NHD", paged=False, chunk_tokens=256, seed=1001)
    if name == "opt13b":
        L = [32768] * 8
        tb, te = _suffix(L, [0.6] * 8)
        return AttnWorkload("opt13b", 8, 40, 40, 128, "f16", L, tb, te, page_size=16, chunk_tokens=512,
                            outlier_frac=0.01, outlier_scale=8.0, seed=1002)
    if name == "opt30b":
        L = [131072] * 4
        tb, te = _suffix(L, [0.5] * 4)
        return AttnWorkload("opt30b", 4, 56, 56, 128, "bf16", L, tb, te, page_size=64, chunk_tokens=2048, seed=1003)
    if name == "llama70b":
        L = [1048576]
        tb, te = _suffix(L, [0.4])
        return AttnWorkload("llama70b", 1, 64, 8, 128, "f16", L, tb, te, page_size=16, chunk_tokens=768,
                            sigma_kv=0.5, seed=1004)
    if name == "ragged":
        key = tensor_key(1005, TENSOR_LENS)
        h = hash64(key, torch.arange(32, dtype=torch.int64))
        u = (_lsr(h, 11).to(torch.float64) / float(1 << 53)).tolist()
        L = [4096 + int(u[i] * (65536 - 4096 + 1)) for i in range(16)]
        shares = [0.1 + 0.8 * u[16 + i] for i in range(16)]
        tb, te = _suffix(L, shares)
        return AttnWorkload("ragged", 16, 32, 8, 128, "f16", L, tb, te, page_size=16, chunk_tokens=512, seed=1005)
    raise KeyError(name)


WORKLOADS = ("tiny", "opt13b", "opt30b", "llama70b", "ragged")


def scaled_down(w: AttnWorkload, factor: int, max_batch: int = 2, max_kv_heads: int = 2) -> AttnWorkload:
    """Same structure (dtype, G, paging, outliers, unaligned suffix slice) at 1/factor the length,
    small enough for the whole-tensor oracle to finish in seconds."""
    B = min(w.B, max_batch)
    Hkv = min(w.Hkv, max_kv_heads)
    L = [max(w.page_size * 2 + 3, l // factor + (7 if l // factor > 64 else 0)) for l in w.seq_lens[:B]]
    tb, te = [], []
    for i in range(B):
        share = (w.tok_end[i] - w.tok_begin[i]) / w.seq_lens[i]
        n = int(share * L[i])
        if w.tok_begin[i] == 0:
            tb.append(0); te.append(n)
        else:
            tb.append(L[i] - n); te.append(L[i])
    return dataclasses.replace(w, name=w.name + "_small", B=B, Hq=Hkv * w.G, Hkv=Hkv, seq_lens=L,
                               tok_begin=tb, tok_end=te, chunk_tokens=min(w.chunk_tokens, 256))

"""ctypes binding of the host-side companions in ``include/hybridgen_host.h`` (argument marshalling only).

Arrays are host torch tensors (16-bit K/V/q as float16 or bfloat16, indices int32, logits float32)."""
from __future__ import annotations

import ctypes as C
from typing import Optional

import torch

from .binding import HG_OK, HgError, _DTYPES, _host, lib

HG_SCHED_POST_QK, HG_SCHED_PRE_QK = 0, 1


class HgHostDesc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32), ("batch", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("dtype", C.c_int32), ("max_selected", C.c_int32), ("num_rows", C.c_int32),
        ("seq_stride", C.c_int64), ("tok_stride", C.c_int64), ("head_stride", C.c_int64), ("scale", C.c_float),
        ("threads", C.c_int32),
    ]


class HgSchedState(C.Structure):
    _fields_ = [("k", C.c_int32), ("strategy", C.c_int32)]


_ready = False


def _lib():
    global _ready
    L = lib()
    if not _ready:
        vp = C.c_void_p
        L.hg_host_logits.argtypes = [vp, vp, vp, vp, vp, C.POINTER(HgHostDesc)]
        L.hg_host_logits.restype = C.c_int
        L.hg_host_select_topk.argtypes = [vp, C.c_int64, C.c_int64, vp, C.c_int32, vp, vp]
        L.hg_host_select_topk.restype = C.c_int
        L.hg_host_group_scores.argtypes = [vp, C.c_int64, C.c_int32, C.c_int64, vp, vp]
        L.hg_host_group_scores.restype = C.c_int
        L.hg_host_gather_logits.argtypes = [vp, C.c_int64, vp, vp, vp, C.POINTER(HgHostDesc)]
        L.hg_host_gather_logits.restype = C.c_int
        L.hg_host_select_positions.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp]
        L.hg_host_select_positions.restype = C.c_int32
        L.hg_host_select_ranked.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, vp, C.c_int32, vp, vp]
        L.hg_host_select_ranked.restype = C.c_int
        L.hg_host_gather_rows.argtypes = [vp, vp, vp, vp, C.POINTER(HgHostDesc)]
        L.hg_host_gather_rows.restype = C.c_int
        L.hg_host_tier_alloc.argtypes = [C.c_size_t, C.c_int32, C.POINTER(vp)]
        L.hg_host_tier_alloc.restype = C.c_int
        L.hg_host_tier_free.argtypes = [vp, C.c_size_t]
        L.hg_host_tier_free.restype = None
        L.hg_host_tier_node_of.argtypes = [vp]
        L.hg_host_tier_node_of.restype = C.c_int32
        L.hg_host_tier_nodes.argtypes = []
        L.hg_host_tier_nodes.restype = C.c_int32
        L.hg_sched_init.argtypes = [C.POINTER(HgSchedState), C.c_int32]
        L.hg_sched_init.restype = None
        L.hg_sched_update.argtypes = [C.POINTER(HgSchedState), C.c_double, C.c_double, C.c_double, C.c_int32, C.c_int32, C.c_int32]
        L.hg_sched_update.restype = None
        _ready = True
    return L


def host_desc(rows: torch.Tensor, num_q_heads: int, max_selected: int, scale: float = 0.0, threads: int = 0) -> HgHostDesc:
    """Describe host rows laid out [B][T][Hkv][D] (any strides with D contiguous)."""
    B, T, Hkv, D = rows.shape
    assert rows.stride(3) == 1
    d = HgHostDesc()
    d.struct_size = C.sizeof(HgHostDesc)
    d.batch, d.num_q_heads, d.num_kv_heads, d.head_dim = B, num_q_heads, Hkv, D
    d.dtype = _DTYPES[rows.dtype]
    d.max_selected = max_selected
    d.num_rows = T
    d.seq_stride, d.tok_stride, d.head_stride = rows.stride(0), rows.stride(1), rows.stride(2)
    d.scale, d.threads = scale, threads
    return d


def _check(st, where):
    if st != HG_OK:
        raise HgError(st, where)


def hg_host_logits(q: torch.Tensor, k_rows: torch.Tensor, idx: Optional[torch.Tensor], n_sel: torch.Tensor,
                   logits: torch.Tensor, desc: HgHostDesc) -> None:
    _check(_lib().hg_host_logits(_host(q, "q"), k_rows.data_ptr(), _host(idx, "idx", torch.int32),
                                 _host(n_sel, "n_sel", torch.int32), _host(logits, "logits", torch.float32), C.byref(desc)),
           "hg_host_logits")


def hg_host_select_topk(scores: torch.Tensor, n: torch.Tensor, k: int):
    rows, stride = scores.shape
    idx = torch.empty(rows, k, dtype=torch.int32)
    n_out = torch.empty(rows, dtype=torch.int32)
    _check(_lib().hg_host_select_topk(_host(scores, "scores", torch.float32), rows, stride, _host(n, "n", torch.int32), k,
                                      idx.data_ptr(), n_out.data_ptr()), "hg_host_select_topk")
    return idx, n_out


def hg_host_group_scores(logits: torch.Tensor, group: int, n: torch.Tensor, scores: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Per-KV-head token scores [rows // group][stride] from per-query-head logits [rows][stride] (group maximum)."""
    rows, stride = logits.shape
    assert rows % group == 0
    if scores is None:
        scores = torch.empty(rows // group, stride)
    _check(_lib().hg_host_group_scores(_host(logits, "logits", torch.float32), rows // group, group, stride,
                                       _host(n, "n", torch.int32), _host(scores, "scores", torch.float32)), "hg_host_group_scores")
    return scores


def hg_host_gather_logits(full: torch.Tensor, idx: torch.Tensor, n_sel: torch.Tensor, out: torch.Tensor, desc: HgHostDesc) -> None:
    """out[b][h][i] = full[b][h][idx[b][h // G][i]] for i < n_sel[b], -inf beyond."""
    _check(_lib().hg_host_gather_logits(_host(full, "full", torch.float32), full.shape[-1], _host(idx, "idx", torch.int32),
                                        _host(n_sel, "n_sel", torch.int32), _host(out, "out", torch.float32), C.byref(desc)),
           "hg_host_gather_logits")


def hg_host_select_positions(n_tokens: int, sinks: int, window: int, k: int) -> torch.Tensor:
    idx = torch.empty(max(k, 1), dtype=torch.int32)
    n = _lib().hg_host_select_positions(n_tokens, sinks, window, k, idx.data_ptr())
    return idx[:n]


def hg_host_select_ranked(ranking: torch.Tensor, n_host: torch.Tensor, k: int):
    """The first K candidates of each (sequence, KV head) list -> (idx [B][Hkv][k] int32, -1 padded; n [B] int32)."""
    B, Hkv, R = ranking.shape
    idx = torch.empty(B, Hkv, k, dtype=torch.int32)
    n = torch.empty(B, dtype=torch.int32)
    _check(_lib().hg_host_select_ranked(_host(ranking, "ranking", torch.int32), B, Hkv, R, _host(n_host, "n_host", torch.int32),
                                        k, idx.data_ptr(), n.data_ptr()), "hg_host_select_ranked")
    return idx, n


def hg_host_gather_rows(rows: torch.Tensor, idx: torch.Tensor, n_sel: torch.Tensor, dst: torch.Tensor, desc: HgHostDesc) -> None:
    _check(_lib().hg_host_gather_rows(rows.data_ptr(), _host(idx, "idx", torch.int32), _host(n_sel, "n_sel", torch.int32),
                                      _host(dst, "dst"), C.byref(desc)), "hg_host_gather_rows")


class FeedbackScheduler:
    """Algorithm 1 as a small controller: feed it the measured stage latencies, read K and the strategy."""

    def __init__(self, k_min: int, k_max: int, step: int):
        self.k_min, self.k_max, self.step = k_min, k_max, step
        self.state = HgSchedState()
        _lib().hg_sched_init(C.byref(self.state), k_min)

    def update(self, t_gpu: float, t_cpu: float, t_tx: float):
        _lib().hg_sched_update(C.byref(self.state), t_gpu, t_cpu, t_tx, self.k_min, self.k_max, self.step)
        return self.state.k, self.state.strategy


def hg_host_tier_nodes() -> int:
    """NUMA nodes with memory on this machine."""
    return int(_lib().hg_host_tier_nodes())


class TierBuffer:
    """A tensor whose memory is bound to one NUMA node (``hg_host_tier_alloc``), optionally registered with the
    CUDA runtime so that copies from and to it are asynchronous DMA.  ``tensor`` views the memory; the buffer
    must outlive every view and every copy in flight."""

    def __init__(self, shape, dtype: torch.dtype, node: int, register: bool = False):
        self.shape, self.dtype, self.node = tuple(shape), dtype, node
        n = 1
        for d in self.shape:
            n *= d
        self.nbytes = max(n * torch.empty(0, dtype=dtype).element_size(), 1)
        ptr = C.c_void_p()
        _check(_lib().hg_host_tier_alloc(self.nbytes, node, C.byref(ptr)), "hg_host_tier_alloc")
        self.ptr = ptr.value
        self._raw = (C.c_uint8 * self.nbytes).from_address(self.ptr)
        self.tensor = torch.frombuffer(self._raw, dtype=dtype, count=n).view(self.shape)
        self.registered = False
        if register:
            err = torch.cuda.cudart().cudaHostRegister(self.ptr, self.nbytes, 0)
            if int(err) != 0:
                self.free()
                raise RuntimeError(f"cudaHostRegister failed: {err}")
            self.registered = True

    def node_of(self, byte_offset: int = 0) -> int:
        return int(_lib().hg_host_tier_node_of(self.ptr + byte_offset))

    def free(self) -> None:
        if self.ptr:
            if self.registered:
                torch.cuda.cudart().cudaHostUnregister(self.ptr)
                self.registered = False
            self.tensor = None
            self._raw = None
            _lib().hg_host_tier_free(self.ptr, self.nbytes)
            self.ptr = 0

    def __del__(self):
        try:
            self.free()
        except Exception:
            pass

"""Thin ctypes binding of the C ABI in ``include/hybridgen_attn.h``.

Only argument marshalling happens here: torch tensors supply device (or host) pointers and the
current CUDA stream; every step of the attention path runs inside the library's kernels.  There is
no fallback: if the library has not been built, or a call returns a non-zero status, an exception
is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_NAME = "libhybridgen_attn.so"
_lib = None

HG_OK, HG_ERR_INVALID_ARG, HG_ERR_UNSUPPORTED, HG_ERR_CUDA, HG_ERR_WORKSPACE = 0, 1, 2, 3, 4
HG_DTYPE_F16, HG_DTYPE_BF16 = 0, 1
HG_DEV_OK, HG_DEV_WAIT_TIMEOUT, HG_DEV_BAD_PAGE, HG_DEV_RANGE = 0, 1, 2, 4
HG_MAX_MERGE_SRC = 8
HG_FLAG_TEST_STALL = 1
HG_FLAG_SPARSE_EMPTY = 2
HG_FLAG_COUNTER_CLEAN = 4
HG_STATIC_SCRATCH_BYTES = 8 << 20
(HG_TUNE_NO_PERSISTENT, HG_TUNE_NO_DYNAMIC, HG_TUNE_NO_PDL, HG_TUNE_NO_MERGE_CLUSTER, HG_TUNE_NO_MERGE_ROWS,
 HG_TUNE_NO_GQA16, HG_TUNE_NO_HOST_DIRECT, HG_TUNE_NO_SPEC_PREFETCH) = 1, 2, 4, 8, 16, 32, 64, 128
HG_LOGITS_TUNE_WARP_MMA, HG_LOGITS_TUNE_TCGEN05 = 1, 2


class HgError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {hg_status_string(status)} (hg_status {status})")


class HgAttnDesc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("batch", C.c_int32),
        ("num_q_heads", C.c_int32),
        ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32),
        ("dtype", C.c_int32),
        ("page_size", C.c_int32),
        ("num_pages", C.c_int32),
        ("page_stride", C.c_int64),
        ("head_stride", C.c_int64),
        ("tok_stride", C.c_int64),
        ("block_table", C.c_void_p),
        ("max_pages", C.c_int32),
        ("chunk_tokens", C.c_int32),
        ("num_chunks", C.c_int32),
        ("scale", C.c_float),
        ("flags", C.c_uint32),
        ("status", C.c_void_p),
        ("sched_counter", C.c_void_p),
        ("tune", C.c_uint32),
        ("tune_stages", C.c_int32),
        ("tune_ctas_per_sm", C.c_int32),
    ]


class HgLogitsDesc(C.Structure):
    _fields_ = [
        ("struct_size", C.c_uint32),
        ("batch", C.c_int32),
        ("num_q_heads", C.c_int32),
        ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32),
        ("dtype", C.c_int32),
        ("max_selected", C.c_int32),
        ("chunk_tokens", C.c_int32),
        ("num_chunks", C.c_int32),
        ("status", C.c_void_p),
        ("tune", C.c_uint32),
        ("reserved", C.c_uint32),
    ]


class HgPartialSrc(C.Structure):
    _fields_ = [("o", C.c_void_p), ("m", C.c_void_p), ("l", C.c_void_p), ("nc", C.c_int32), ("reserved", C.c_int32)]


def lib_path() -> str:
    return os.path.join(_PKG, _LIB_NAME)


def lib():
    """Load the CUDA library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        path = lib_path()
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: build it with `python -m paper_2604_18529_b200.build` "
                               "(there is no CPU or PyTorch fallback)")
        L = C.CDLL(path)
        vp, i32 = C.c_void_p, C.c_int32
        L.hg_attn_partial.argtypes = [vp] * 10 + [C.POINTER(HgAttnDesc)]
        L.hg_attn_partial.restype = C.c_int
        L.hg_attn_merge.argtypes = [C.POINTER(HgPartialSrc), i32, vp, vp, vp, C.POINTER(HgAttnDesc)]
        L.hg_attn_merge.restype = C.c_int
        L.hg_attn_workspace_bytes.argtypes = [C.POINTER(HgAttnDesc), i32]
        L.hg_attn_workspace_bytes.restype = C.c_size_t
        L.hg_attn_decode.argtypes = [vp] * 6 + [C.POINTER(HgPartialSrc), i32, vp, vp, vp, C.c_size_t, vp, C.POINTER(HgAttnDesc)]
        L.hg_attn_decode.restype = C.c_int
        L.hg_attn_decode_host.argtypes = L.hg_attn_decode.argtypes
        L.hg_attn_decode_host.restype = C.c_int
        L.hg_attn_decode_static.argtypes = [vp] * 6 + [C.POINTER(HgPartialSrc), i32, vp, vp, vp, C.POINTER(HgAttnDesc)]
        L.hg_attn_decode_static.restype = C.c_int
        L.hg_attn_partial_from_logits.argtypes = [vp] * 7 + [C.POINTER(HgLogitsDesc)]
        L.hg_attn_partial_from_logits.restype = C.c_int
        L.hg_kv_append.argtypes = [vp] * 7 + [C.POINTER(HgAttnDesc)]
        L.hg_kv_append.restype = C.c_int
        L.hg_kv_evict.argtypes = [vp] * 5 + [i32, vp, vp, vp, vp, i32, vp, C.POINTER(HgAttnDesc)]
        L.hg_kv_evict.restype = C.c_int
        L.hg_kv_evict_begin.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, C.POINTER(HgAttnDesc)]
        L.hg_kv_evict_begin.restype = C.c_int
        L.hg_kv_evict_copy.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp, C.POINTER(HgAttnDesc)]
        L.hg_kv_evict_copy.restype = C.c_int
        L.hg_kv_evict_finish.argtypes = [vp, vp, vp, vp, i32, vp, C.POINTER(HgAttnDesc)]
        L.hg_kv_evict_finish.restype = C.c_int
        L.hg_kv_read_probe.argtypes = [vp] * 7 + [C.POINTER(HgAttnDesc)]
        L.hg_kv_read_probe.restype = C.c_int
        L.hg_status_string.argtypes = [C.c_int]
        L.hg_status_string.restype = C.c_char_p
        L.hg_version.argtypes = []
        L.hg_version.restype = C.c_uint32
        _lib = L
    return _lib


def hg_status_string(status: int) -> str:
    return lib().hg_status_string(int(status)).decode()


def hg_version() -> int:
    return int(lib().hg_version())


def _dev(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must be a CUDA tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _host(t: Optional[torch.Tensor], name: str, dtype=None) -> Optional[int]:
    if t is None:
        return None
    if t.is_cuda:
        raise ValueError(f"{name} must be a host tensor")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"{name} must be {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _check(status: int, where: str) -> None:
    if status != HG_OK:
        raise HgError(status, where)


_DTYPES = {torch.float16: HG_DTYPE_F16, torch.bfloat16: HG_DTYPE_BF16, "f16": HG_DTYPE_F16, "bf16": HG_DTYPE_BF16}


def attn_desc(*, batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, dtype, page_size: int,
              num_pages: int, page_stride: int, head_stride: int, tok_stride: int,
              block_table: Optional[torch.Tensor], max_pages: int, chunk_tokens: int, num_chunks: int,
              scale: float = 0.0, status: Optional[torch.Tensor] = None, flags: int = 0,
              sched_counter: Optional[torch.Tensor] = None, tune: int = 0, tune_stages: int = 0,
              tune_ctas_per_sm: int = 0) -> HgAttnDesc:
    """Fill an ``hg_attn_desc``.  ``block_table`` (int32 CUDA [B][max_pages]), ``status`` and
    ``sched_counter`` (int32 CUDA scalars) are kept alive by the returned object."""
    d = HgAttnDesc()
    d.struct_size = C.sizeof(HgAttnDesc)
    d.batch, d.num_q_heads, d.num_kv_heads, d.head_dim = batch, num_q_heads, num_kv_heads, head_dim
    d.dtype = _DTYPES[dtype]
    d.page_size, d.num_pages = page_size, num_pages
    d.page_stride, d.head_stride, d.tok_stride = page_stride, head_stride, tok_stride
    d.block_table = _dev(block_table, "block_table", torch.int32)
    d.max_pages, d.chunk_tokens, d.num_chunks = max_pages, chunk_tokens, num_chunks
    d.scale, d.flags = scale, flags
    d.status = _dev(status, "status", torch.int32)
    d.sched_counter = _dev(sched_counter, "sched_counter", torch.int32)
    d.tune, d.tune_stages, d.tune_ctas_per_sm = tune, tune_stages, tune_ctas_per_sm
    d._keep = (block_table, status, sched_counter)
    return d


def _src_array(partials: Sequence[Tuple[torch.Tensor, torch.Tensor, torch.Tensor]], host: bool):
    arr = (HgPartialSrc * max(1, len(partials)))()
    conv = _host if host else _dev
    for i, (o, m, l) in enumerate(partials):
        arr[i].o = conv(o, "partial o", torch.float32)
        arr[i].m = conv(m, "partial m", torch.float32)
        arr[i].l = conv(l, "partial l", torch.float32)
        arr[i].nc = m.shape[-1]
        if o.numel() != m.numel() * o.shape[-1] or l.shape != m.shape:
            raise ValueError("partial source shapes must be o [B][Hq][nc][D], m and l [B][Hq][nc]")
    return arr


def hg_attn_partial(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, o_part, m_part, l_part, desc: HgAttnDesc,
                    stream=None) -> None:
    """Chunk partials (o, m, l) of the GPU-resident slice; see ``hg_attn_partial`` in the header."""
    st = lib().hg_attn_partial(_dev(q, "q"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                               _dev(seq_lens, "seq_lens", torch.int32), _dev(tok_begin, "tok_begin", torch.int32),
                               _dev(tok_end, "tok_end", torch.int32), _dev(o_part, "o_part", torch.float32),
                               _dev(m_part, "m_part", torch.float32), _dev(l_part, "l_part", torch.float32),
                               _stream(stream), C.byref(desc))
    _check(st, "hg_attn_partial")


def logits_desc(*, batch: int, num_q_heads: int, num_kv_heads: int, head_dim: int, dtype, max_selected: int,
                chunk_tokens: int = 256, num_chunks: int = 0, status: Optional[torch.Tensor] = None,
                tune: int = 0) -> HgLogitsDesc:
    d = HgLogitsDesc()
    d.struct_size = C.sizeof(HgLogitsDesc)
    d.batch, d.num_q_heads, d.num_kv_heads, d.head_dim = batch, num_q_heads, num_kv_heads, head_dim
    d.dtype = _DTYPES[dtype]
    d.max_selected, d.chunk_tokens = max_selected, chunk_tokens
    d.num_chunks = num_chunks or -(-max_selected // chunk_tokens)
    d.status = _dev(status, "status", torch.int32)
    d.tune = tune
    d._keep = (status,)
    return d


def hg_attn_partial_from_logits(logits, v_rows, n_sel, o_part, m_part, l_part, desc: HgLogitsDesc, stream=None) -> None:
    """Partials (o, m, l) from host-computed logits [B][Hq][K] (fp32) and the matching V rows [B][Hkv][K][D]."""
    st = lib().hg_attn_partial_from_logits(_dev(logits, "logits", torch.float32), _dev(v_rows, "v_rows"),
                                           _dev(n_sel, "n_sel", torch.int32), _dev(o_part, "o_part", torch.float32),
                                           _dev(m_part, "m_part", torch.float32), _dev(l_part, "l_part", torch.float32),
                                           _stream(stream), C.byref(desc))
    _check(st, "hg_attn_partial_from_logits")


def hg_attn_merge(partials, out, lse, desc: HgAttnDesc, stream=None) -> None:
    """LSE-merge of partial sources [(o, m, l), ...] (device tensors) into out [B][Hq][D] and lse [B][Hq]."""
    arr = _src_array(partials, host=False)
    st = lib().hg_attn_merge(arr, len(partials), _dev(out, "out", torch.float32), _dev(lse, "lse", torch.float32),
                             _stream(stream), C.byref(desc))
    _check(st, "hg_attn_merge")


def hg_attn_suggest_chunk(total_tokens: int, num_q_heads: int, num_kv_heads: int, page_size: int) -> int:
    """A chunk size (tokens) for a problem with that many GPU-resident token positions in total."""
    f = lib().hg_attn_suggest_chunk
    f.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_int32]
    f.restype = C.c_int32
    n = int(f(total_tokens, num_q_heads, num_kv_heads, page_size))
    if n == 0:
        raise HgError(HG_ERR_INVALID_ARG, "hg_attn_suggest_chunk")
    return n


def hg_attn_workspace_bytes(desc: HgAttnDesc, n_host_partials: int = 0) -> int:
    n = int(lib().hg_attn_workspace_bytes(C.byref(desc), n_host_partials))
    if n == 0:
        raise HgError(HG_ERR_INVALID_ARG, "hg_attn_workspace_bytes")
    return n


def hg_attn_decode(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, host_partials, out, lse, workspace,
                   desc: HgAttnDesc, stream=None) -> None:
    """partial + merge in one call; ``host_partials`` are device tensors holding the host-slice partials."""
    arr = _src_array(host_partials, host=False)
    st = lib().hg_attn_decode(_dev(q, "q"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                              _dev(seq_lens, "seq_lens", torch.int32), _dev(tok_begin, "tok_begin", torch.int32),
                              _dev(tok_end, "tok_end", torch.int32), arr, len(host_partials),
                              _dev(out, "out", torch.float32), _dev(lse, "lse", torch.float32),
                              _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                              _stream(stream), C.byref(desc))
    _check(st, "hg_attn_decode")


def hg_attn_decode_static(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, host_partials, out, lse,
                          desc: HgAttnDesc, stream=None) -> None:
    """``hg_attn_decode`` for callers that may not allocate device memory (fixed-budget plugins,
    allocator-free decode loops, components without an allocator): the chunk partials go to a fixed 8 MiB array inside the
    library instead of a caller workspace.  Raises ``HgError`` (workspace) if the problem's partials do
    not fit.  All calls on a device share that array, so calls that could overlap on the GPU must be
    serialised; make the first call on a device outside any stream capture."""
    arr = _src_array(host_partials, host=False)
    st = lib().hg_attn_decode_static(_dev(q, "q"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                                     _dev(seq_lens, "seq_lens", torch.int32), _dev(tok_begin, "tok_begin", torch.int32),
                                     _dev(tok_end, "tok_end", torch.int32), arr, len(host_partials),
                                     _dev(out, "out", torch.float32), _dev(lse, "lse", torch.float32),
                                     _stream(stream), C.byref(desc))
    _check(st, "hg_attn_decode_static")


def hg_attn_decode_host(q_host, k_cache, v_cache, seq_lens_host, tok_begin_host, tok_end_host, host_partials_host,
                        out_host, lse_host, workspace, desc: HgAttnDesc, stream=None) -> None:
    """The same pass with per-step data in host (ideally pinned) memory; results land in out_host / lse_host
    once the stream has been synchronised."""
    arr = _src_array(host_partials_host, host=True)
    st = lib().hg_attn_decode_host(_host(q_host, "q_host"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                                   _host(seq_lens_host, "seq_lens_host", torch.int32),
                                   _host(tok_begin_host, "tok_begin_host", torch.int32),
                                   _host(tok_end_host, "tok_end_host", torch.int32), arr, len(host_partials_host),
                                   _host(out_host, "out_host", torch.float32), _host(lse_host, "lse_host", torch.float32),
                                   _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(),
                                   _stream(stream), C.byref(desc))
    _check(st, "hg_attn_decode_host")


def _prepared(fn, args, keep, where: str):
    def call(_keep=keep) -> None:
        st = fn(*args)
        if st != HG_OK:
            _check(st, where)
    return call


def prepare_partial(q, k_cache, v_cache, seq_lens, tok_begin, tok_end, o_part, m_part, l_part, desc: HgAttnDesc, stream=None):
    """``hg_attn_partial`` with its arguments marshalled once: returns a callable for a decode loop that reuses the
    same buffers (and stream) every step.  The callable keeps the tensors alive."""
    args = (_dev(q, "q"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"), _dev(seq_lens, "seq_lens", torch.int32),
            _dev(tok_begin, "tok_begin", torch.int32), _dev(tok_end, "tok_end", torch.int32),
            _dev(o_part, "o_part", torch.float32), _dev(m_part, "m_part", torch.float32), _dev(l_part, "l_part", torch.float32),
            _stream(stream), C.byref(desc))
    keep = (q, k_cache, v_cache, seq_lens, tok_begin, tok_end, o_part, m_part, l_part, desc)
    return _prepared(lib().hg_attn_partial, args, keep, "hg_attn_partial")


def prepare_merge(partials, out, lse, desc: HgAttnDesc, stream=None):
    """``hg_attn_merge`` with its arguments marshalled once (see ``prepare_partial``)."""
    arr = _src_array(partials, host=False)
    args = (arr, len(partials), _dev(out, "out", torch.float32), _dev(lse, "lse", torch.float32), _stream(stream), C.byref(desc))
    return _prepared(lib().hg_attn_merge, args, (partials, out, lse, desc, arr), "hg_attn_merge")


def prepare_decode_host(q_host, k_cache, v_cache, seq_lens_host, tok_begin_host, tok_end_host, host_partials_host,
                        out_host, lse_host, workspace, desc: HgAttnDesc, stream=None):
    """Marshal the arguments of ``hg_attn_decode_host`` once and return a callable that makes the call.

    For a decode loop that reuses the same buffers every step (the usual case): the per-call cost of
    checking and converting a dozen tensors is paid once.  The returned callable keeps the tensors alive.
    """
    arr = _src_array(host_partials_host, host=True)
    args = (_host(q_host, "q_host"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
            _host(seq_lens_host, "seq_lens_host", torch.int32), _host(tok_begin_host, "tok_begin_host", torch.int32),
            _host(tok_end_host, "tok_end_host", torch.int32), arr, len(host_partials_host),
            _host(out_host, "out_host", torch.float32), _host(lse_host, "lse_host", torch.float32),
            _dev(workspace, "workspace"), workspace.numel() * workspace.element_size(), _stream(stream), C.byref(desc))
    keep = (q_host, k_cache, v_cache, seq_lens_host, tok_begin_host, tok_end_host, host_partials_host, out_host, lse_host,
            workspace, desc, arr)
    return _prepared(lib().hg_attn_decode_host, args, keep, "hg_attn_decode_host")


def hg_kv_append(k_new, v_new, k_cache, v_cache, seq_lens, tok_end, desc: HgAttnDesc, stream=None) -> None:
    """Write this step's K/V rows [B][Hkv][D] at position seq_lens[b] and advance seq_lens (and tok_end)."""
    st = lib().hg_kv_append(_dev(k_new, "k_new"), _dev(v_new, "v_new"), _dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                            _dev(seq_lens, "seq_lens", torch.int32), _dev(tok_end, "tok_end", torch.int32),
                            _stream(stream), C.byref(desc))
    _check(st, "hg_kv_append")


def hg_kv_evict(k_cache, v_cache, tok_begin, tok_end, n_evict, k_out, v_out, freed_pages, n_freed, desc: HgAttnDesc,
                stream=None) -> None:
    """Copy the oldest n_evict[b] tokens of every slice to k_out / v_out [B][max_evict][Hkv][D], advance tok_begin
    and un-map the pages that became empty (their ids go to freed_pages [B][max_freed])."""
    st = lib().hg_kv_evict(_dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"), _dev(tok_begin, "tok_begin", torch.int32),
                           _dev(tok_end, "tok_end", torch.int32), _dev(n_evict, "n_evict", torch.int32), k_out.shape[1],
                           _dev(k_out, "k_out"), _dev(v_out, "v_out"), _dev(freed_pages, "freed_pages", torch.int32),
                           _dev(n_freed, "n_freed", torch.int32), 0 if freed_pages is None else freed_pages.shape[1],
                           _stream(stream), C.byref(desc))
    _check(st, "hg_kv_evict")


def hg_kv_evict_begin(tok_begin, tok_end, n_evict, max_evict: int, max_freed: int, src_begin, n_moved, desc: HgAttnDesc,
                      stream=None) -> None:
    """Step 1 of an eviction that drains beside the attention: decide and record the rows that leave, advance tok_begin."""
    st = lib().hg_kv_evict_begin(_dev(tok_begin, "tok_begin", torch.int32), _dev(tok_end, "tok_end", torch.int32),
                                 _dev(n_evict, "n_evict", torch.int32), max_evict, max_freed,
                                 _dev(src_begin, "src_begin", torch.int32), _dev(n_moved, "n_moved", torch.int32),
                                 _stream(stream), C.byref(desc))
    _check(st, "hg_kv_evict_begin")


def hg_kv_evict_copy(k_cache, v_cache, src_begin, n_moved, k_out, v_out, desc: HgAttnDesc, stream=None) -> None:
    """Step 2: copy the recorded rows to k_out / v_out [B][max_evict][Hkv][D] (reads only)."""
    st = lib().hg_kv_evict_copy(_dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"), _dev(src_begin, "src_begin", torch.int32),
                                _dev(n_moved, "n_moved", torch.int32), k_out.shape[1], _dev(k_out, "k_out"),
                                _dev(v_out, "v_out"), _stream(stream), C.byref(desc))
    _check(st, "hg_kv_evict_copy")


def hg_kv_evict_finish(src_begin, n_moved, freed_pages, n_freed, desc: HgAttnDesc, stream=None) -> None:
    """Step 3: un-map and list the pages that lie wholly below the new beginning."""
    st = lib().hg_kv_evict_finish(_dev(src_begin, "src_begin", torch.int32), _dev(n_moved, "n_moved", torch.int32),
                                  _dev(freed_pages, "freed_pages", torch.int32), _dev(n_freed, "n_freed", torch.int32),
                                  0 if freed_pages is None else freed_pages.shape[1], _stream(stream), C.byref(desc))
    _check(st, "hg_kv_evict_finish")


def hg_kv_read_probe(k_cache, v_cache, seq_lens, tok_begin, tok_end, sink, desc: HgAttnDesc, stream=None) -> None:
    """Stream the slice's K and V tiles and XOR-fold them into sink [B][Hkv][NC] (uint32 viewed as int32)."""
    st = lib().hg_kv_read_probe(_dev(k_cache, "k_cache"), _dev(v_cache, "v_cache"),
                                _dev(seq_lens, "seq_lens", torch.int32), _dev(tok_begin, "tok_begin", torch.int32),
                                _dev(tok_end, "tok_end", torch.int32), _dev(sink, "sink", torch.int32),
                                _stream(stream), C.byref(desc))
    _check(st, "hg_kv_read_probe")

"""The C-ABI library without a GPU: it loads, exports every symbol the header declares, and rejects
bad arguments before touching CUDA.  No compute calls here."""
import ctypes as C
import os
import re

import pytest

import paper_2604_18529_b200 as pkg
from paper_2604_18529_b200 import binding as hg
from paper_2604_18529_b200 import build as hgbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
HEADERS = [os.path.join(ROOT, "include", "hybridgen_attn.h"), os.path.join(ROOT, "include", "hybridgen_host.h")]


@pytest.fixture(scope="module")
def lib():
    hgbuild.build()
    return hg.lib()


def declared_functions():
    names = set()
    for header in HEADERS:
        src = re.sub(r"/\*.*?\*/", "", open(header).read(), flags=re.S)
        names |= set(re.findall(r"\b(hg_[a-z_0-9]+)\s*\(", src))
    return sorted(names)


def test_header_functions_are_exported(lib):
    names = declared_functions()
    assert {"hg_attn_partial", "hg_attn_merge", "hg_attn_decode", "hg_attn_decode_host",
            "hg_attn_workspace_bytes", "hg_kv_read_probe", "hg_status_string", "hg_version", "hg_attn_decode_static",
            "hg_attn_partial_from_logits", "hg_host_logits", "hg_host_select_topk", "hg_host_select_positions",
            "hg_host_gather_rows", "hg_sched_init", "hg_sched_update"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_version_and_status_strings(lib):
    assert pkg.hg_version() == 0x00010000
    assert pkg.hg_status_string(0) == "ok"
    assert "invalid" in pkg.hg_status_string(1)
    assert "unsupported" in pkg.hg_status_string(2)
    assert "unknown" in pkg.hg_status_string(99)


def test_desc_struct_matches_the_c_layout():
    # offsets follow natural C alignment of the header's field order
    f = {n: getattr(hg.HgAttnDesc, n).offset for n, _ in hg.HgAttnDesc._fields_}
    assert f["struct_size"] == 0 and f["num_pages"] == 28 and f["page_stride"] == 32 and f["block_table"] == 56
    assert f["max_pages"] == 64 and f["flags"] == 80 and f["status"] == 88 and f["sched_counter"] == 96
    assert f["tune"] == 104 and f["tune_stages"] == 108 and f["tune_ctas_per_sm"] == 112
    assert C.sizeof(hg.HgAttnDesc) == 120
    assert C.sizeof(hg.HgPartialSrc) == 32


def good_desc(**over):
    kw = dict(batch=2, num_q_heads=8, num_kv_heads=2, head_dim=128, dtype="f16", page_size=16, num_pages=64,
              page_stride=2 * 16 * 128, head_stride=16 * 128, tok_stride=128, block_table=None, max_pages=32,
              chunk_tokens=256, num_chunks=2)
    kw.update(over)
    return hg.attn_desc(**kw)


FAKE = 0x10000  # a non-null, 16-byte aligned address; never dereferenced because validation fails first


def call_partial(lib, d, **ptr):
    a = dict(q=FAKE, k=FAKE, v=FAKE, sl=FAKE, tb=FAKE, te=FAKE, o=FAKE, m=FAKE, l=FAKE)
    a.update(ptr)
    return lib.hg_attn_partial(a["q"], a["k"], a["v"], a["sl"], a["tb"], a["te"], a["o"], a["m"], a["l"], None, C.byref(d))


@pytest.mark.parametrize("over,want", [
    (dict(batch=0), hg.HG_ERR_INVALID_ARG),
    (dict(num_q_heads=6, num_kv_heads=4), hg.HG_ERR_INVALID_ARG),
    (dict(head_dim=96), hg.HG_ERR_UNSUPPORTED),
    (dict(head_dim=100), hg.HG_ERR_INVALID_ARG),
    (dict(page_size=24), hg.HG_ERR_UNSUPPORTED),
    (dict(page_size=8), hg.HG_ERR_UNSUPPORTED),
    (dict(tok_stride=132), hg.HG_ERR_INVALID_ARG),
    (dict(tok_stride=64), hg.HG_ERR_INVALID_ARG),
    (dict(chunk_tokens=96), hg.HG_ERR_UNSUPPORTED),
    (dict(chunk_tokens=0), hg.HG_ERR_INVALID_ARG),
    (dict(chunk_tokens=32768, page_size=16), hg.HG_ERR_UNSUPPORTED),
    (dict(num_chunks=0), hg.HG_ERR_INVALID_ARG),
    (dict(scale=-1.0), hg.HG_ERR_INVALID_ARG),
    (dict(num_pages=10), hg.HG_ERR_INVALID_ARG),          # identity paging needs batch * max_pages pages
])
def test_partial_rejects_bad_descriptions(lib, over, want):
    assert call_partial(lib, good_desc(**over)) == want


def test_partial_rejects_null_misaligned_and_short_struct(lib):
    d = good_desc()
    for k in ("q", "k", "v", "sl", "tb", "te", "o", "m", "l"):
        assert call_partial(lib, d, **{k: None}) == hg.HG_ERR_INVALID_ARG, k
    assert call_partial(lib, d, k=FAKE + 8) == hg.HG_ERR_INVALID_ARG
    assert call_partial(lib, d, q=FAKE + 2) == hg.HG_ERR_INVALID_ARG
    d.struct_size = 8
    assert call_partial(lib, d) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_partial(FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE, None, None) == hg.HG_ERR_INVALID_ARG


def test_merge_and_decode_reject_bad_arguments(lib):
    d = good_desc()
    src = (hg.HgPartialSrc * 2)()
    src[0].o, src[0].m, src[0].l, src[0].nc = FAKE, FAKE, FAKE, 1
    assert lib.hg_attn_merge(src, 0, FAKE, FAKE, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_merge(src, 9, FAKE, FAKE, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_merge(None, 1, FAKE, FAKE, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_merge(src, 1, None, FAKE, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_merge(src, 2, FAKE, FAKE, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG   # second source is null
    src[0].nc = 0
    assert lib.hg_attn_merge(src, 1, FAKE, FAKE, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    src[0].nc = 1
    # workspace: missing, misaligned, too small
    args = [FAKE] * 6 + [src, 1, FAKE, FAKE]
    assert lib.hg_attn_decode(*args, None, 1 << 30, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_decode(*args, FAKE + 16, 1 << 30, None, C.byref(d)) == hg.HG_ERR_INVALID_ARG
    assert lib.hg_attn_decode(*args, FAKE, 1024, None, C.byref(d)) == hg.HG_ERR_WORKSPACE
    assert lib.hg_attn_decode_host(*args, FAKE, 1024, None, C.byref(d)) == hg.HG_ERR_WORKSPACE


def test_shorter_struct_without_the_trailing_field_is_accepted(lib):
    d = good_desc()
    d.struct_size = 96                       # a caller compiled before sched_counter existed
    d.sched_counter = 0x3                    # garbage behind the declared size must be ignored
    assert call_partial(lib, d, q=None) == hg.HG_ERR_INVALID_ARG      # gets as far as the pointer checks
    d.struct_size = 104                      # a caller compiled before the tuning fields existed
    assert call_partial(lib, d) == hg.HG_ERR_INVALID_ARG              # now the misaligned counter is seen
    d.sched_counter = 0
    d.tune, d.tune_stages, d.tune_ctas_per_sm = 0xffffffff, 99, -5   # behind the declared size: ignored
    assert call_partial(lib, d, q=None) == hg.HG_ERR_INVALID_ARG


def test_workspace_bytes(lib):
    d = good_desc()
    rows = 2 * 8
    need = rows * 2 * 128 * 4 + 2 * rows * 2 * 4      # chunk partials alone
    n0 = pkg.hg_attn_workspace_bytes(d, 0)
    n2 = pkg.hg_attn_workspace_bytes(d, 2)
    assert n0 >= need and n2 >= n0 + rows * 2 * 130 * 4
    assert n0 % 256 == 0
    with pytest.raises(hg.HgError):
        pkg.hg_attn_workspace_bytes(good_desc(head_dim=96), 0)


def test_binding_refuses_host_tensors_for_device_arguments():
    import torch
    d = good_desc()
    t = torch.zeros(4)
    with pytest.raises(ValueError):
        pkg.hg_attn_partial(t, t, t, t, t, t, t, t, t, d, stream=0)


def test_suggested_chunk_is_always_a_legal_one():
    import paper_2604_18529_b200 as pkg
    for page in (16, 32, 64, 128, 256):
        for tokens in (0, 1, 1000, 157_280, 419_430, 10**9):
            for hq, hkv in ((8, 8), (32, 8), (64, 8), (64, 4), (96, 8)):
                c = pkg.hg_attn_suggest_chunk(tokens, hq, hkv, page)
                assert c % 64 == 0 and c % page == 0 and max(128, page) <= c <= 1024
    assert pkg.hg_attn_suggest_chunk(2048, 64, 8, 16) == 128           # a small problem is cut fine
    assert pkg.hg_attn_suggest_chunk(10**7, 64, 8, 16) == 1024          # a large one coarse
    assert pkg.hg_attn_suggest_chunk(278_000, 32, 8, 16) == 512 and pkg.hg_attn_suggest_chunk(419_430, 64, 8, 16) == 768
    for bad in ((-1, 8, 8, 16), (100, 8, 3, 16), (100, 8, 8, 48), (100, 0, 1, 16)):
        with pytest.raises(pkg.HgError):
            pkg.hg_attn_suggest_chunk(*bad)

"""B200-native decode attention over the GPU-resident slice of a long KV cache:
per-chunk softmax partials (``hg_attn_partial``) and their log-sum-exp merge with
partials for the host-held slice (``hg_attn_merge``).

The arithmetic runs in the CUDA library under ``csrc/``; this package only marshals
arguments. Importing it does not load the library; the first call does, and raises if
the library has not been built.
"""
from .binding import (  # noqa: F401
    HgError,
    lib,
    lib_path,
    attn_desc,
    hg_attn_partial,
    hg_attn_merge,
    hg_attn_partial_from_logits,
    logits_desc,
    hg_attn_decode,
    hg_attn_decode_host,
    prepare_decode_host,
    prepare_merge,
    prepare_partial,
    hg_attn_decode_static,
    hg_attn_suggest_chunk,
    hg_attn_workspace_bytes,
    hg_status_string,
    hg_kv_read_probe,
    hg_kv_append,
    hg_kv_evict,
    hg_kv_evict_begin,
    hg_kv_evict_copy,
    hg_kv_evict_finish,
    hg_version,
)

"""Pins for the fp64 oracle against things other than itself: brute force written another way,
library float types, closed forms, invariants the paper states, and a hand-worked example.
CPU only."""
import math
import os

import numpy as np
import pytest

from oracle import hg_oracle as O

RNG = np.random.default_rng(20260418)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


def f16_bits(x):
    return np.asarray(x, dtype=np.float16).view(np.uint16)


def bf16_bits(x):
    """Round-to-nearest-even fp32 -> bf16 bit patterns (integer arithmetic, written for the test)."""
    u = np.asarray(x, dtype=np.float32).view(np.uint32).astype(np.uint64)
    u = u + 0x7FFF + ((u >> 16) & 1)
    return (u >> 16).astype(np.uint16)


def np_decode(bits, dtype):
    """Library decode: numpy's own half type; bf16 as the upper half of an IEEE fp32."""
    bits = np.asarray(bits, dtype=np.uint16)
    if dtype == "f16":
        return bits.view(np.float16).astype(np.longdouble)
    return (bits.astype(np.uint32) << 16).view(np.float32).astype(np.longdouble)


def enc(x, dtype):
    return f16_bits(x) if dtype == "f16" else bf16_bits(x)


def brute(q, K, V, dtype, tokens, scale=None):
    """Direct softmax attention in long double on explicitly gathered arrays."""
    qd, Kd, Vd = np_decode(q, dtype), np_decode(K, dtype)[tokens], np_decode(V, dtype)[tokens]
    D = qd.shape[-1]
    s = (Kd * qd[None, :]).sum(axis=1) * (np.longdouble(1) / np.sqrt(np.longdouble(D)) if scale is None else scale)
    w = np.exp(s)
    out = (w[:, None] * Vd).sum(axis=0) / w.sum()
    return out.astype(np.float64), float(np.log(w.sum())), s.astype(np.float64)


def rand_case(n, D, dtype, sigma=1.0):
    q = enc(RNG.standard_normal(D), dtype)
    K = enc(RNG.standard_normal((n, D)) * sigma, dtype)
    V = enc(RNG.standard_normal((n, D)) * sigma, dtype)
    return q, K, V


# ---- codecs ---------------------------------------------------------------------------------

def test_decode_named_patterns():
    L = O.lib()
    assert L.hgo_decode_f16(0x3C00) == 1.0
    assert L.hgo_decode_f16(0x7BFF) == 65504.0
    assert L.hgo_decode_f16(0x0001) == 2.0 ** -24
    assert L.hgo_decode_f16(0xFC00) == -math.inf
    assert L.hgo_decode_f16(0xC000) == -2.0
    assert L.hgo_decode_bf16(0x3F80) == 1.0
    assert L.hgo_decode_bf16(0x0080) == 2.0 ** -126
    assert L.hgo_decode_bf16(0x0001) == 2.0 ** -133
    assert L.hgo_decode_bf16(0xC040) == -3.0


@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_decode_all_patterns_match_library_types(dtype):
    bits = np.arange(65536, dtype=np.uint16)
    mine = O.decode(bits, dtype)
    ref = np_decode(bits, dtype).astype(np.float64)
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(mine), nan)
    assert np.array_equal(mine[~nan], ref[~nan])
    assert np.array_equal(np.signbit(mine[~nan]), np.signbit(ref[~nan]))


# ---- brute force on tiny inputs ----------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f16", "bf16"])
@pytest.mark.parametrize("n,D", [(1, 2), (2, 4), (5, 8), (33, 8), (17, 64)])
def test_full_matches_brute_force(dtype, n, D):
    q, K, V = rand_case(n, D, dtype)
    out, lse = O.full(q, K, V, dtype)
    bo, bl, bs = brute(q, K, V, dtype, np.arange(n))
    np.testing.assert_allclose(out, bo, rtol=0, atol=1e-13)
    assert abs(lse - bl) < 1e-13
    np.testing.assert_allclose(O.logits(q, K, dtype), bs, rtol=0, atol=1e-13)


def test_logits_scale_and_operand_roles():
    """s_t = <q, K_t>/sqrt(D): catches a transposed operand, a wrong stride, a missing or squared scale."""
    D, n = 16, 7
    q = f16_bits(np.arange(1, D + 1) / 8.0)
    K = f16_bits((np.arange(n)[:, None] * 2.0 + np.arange(D)[None, :] % 3) / 4.0)
    s = O.logits(q, K, "f16")
    want = [sum((d + 1) / 8.0 * ((t * 2.0 + d % 3) / 4.0) for d in range(D)) / 4.0 for t in range(n)]
    np.testing.assert_allclose(s, want, rtol=0, atol=1e-14)
    np.testing.assert_allclose(O.logits(q, K, "f16", scale=0.5), np.asarray(want) * 2.0, atol=1e-14)
    # token subset through an index list and through a range give the same rows
    np.testing.assert_allclose(O.logits(q, K, "f16", idx=[5, 1]), [want[5], want[1]], atol=1e-14)
    np.testing.assert_allclose(O.logits(q, K, "f16", t0=2, n=3), want[2:5], atol=1e-14)


# ---- the paper's exactness claim: any token split merges back to monolithic attention -----------

@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_merge_of_partials_equals_full_for_every_split_point(dtype):
    n, D = 41, 8
    q, K, V = rand_case(n, D, dtype, sigma=2.0)
    out, lse = O.full(q, K, V, dtype)
    for cut in range(n + 1):
        a = O.partial(q, K, V, dtype, t0=0, n=cut)
        b = O.partial(q, K, V, dtype, t0=cut, n=n - cut)
        mo, ml = O.merge([a[0], b[0]], [a[1], b[1]], [a[2], b[2]])
        np.testing.assert_allclose(mo, out, rtol=1e-12, atol=1e-14)
        assert abs(ml - lse) < 1e-12


@pytest.mark.parametrize("chunk", [1, 7, 16, 2048])
def test_merge_of_chunk_partials_equals_full(chunk):
    n, D = 300, 16
    q, K, V = rand_case(n, D, "f16", sigma=1.5)
    out, lse = O.full(q, K, V, "f16")
    parts = [O.partial(q, K, V, "f16", t0=a, n=min(chunk, n - a)) for a in range(0, n, chunk)]
    parts.append(O.partial(q, K, V, "f16", t0=0, n=0))            # an empty source changes nothing
    mo, ml = O.merge([p[0] for p in parts], [p[1] for p in parts], [p[2] for p in parts])
    np.testing.assert_allclose(mo, out, rtol=1e-12, atol=1e-14)
    assert abs(ml - lse) < 1e-12


def test_literal_concatenation_equals_full_and_merge():
    n, D = 57, 8
    q, K, V = rand_case(n, D, "bf16")
    out, lse = O.full(q, K, V, "bf16")
    perm = RNG.permutation(n)
    for cut in (0, 1, 20, n):
        A, B = np.sort(perm[:cut]), np.sort(perm[cut:])          # interleaved, not contiguous, sets
        lo, ll = O.literal(q, K, V, "bf16", A, B)
        np.testing.assert_allclose(lo, out, rtol=1e-12, atol=1e-14)
        assert abs(ll - lse) < 1e-12
        pa, pb = O.partial(q, K, V, "bf16", idx=A), O.partial(q, K, V, "bf16", idx=B)
        mo, ml = O.merge([pa[0], pb[0]], [pa[1], pb[1]], [pa[2], pb[2]])
        np.testing.assert_allclose(mo, lo, rtol=1e-12, atol=1e-14)
        assert abs(ml - ll) < 1e-12


def test_empty_sets():
    q, K, V = rand_case(4, 8, "f16")
    m, l, o = O.partial(q, K, V, "f16", t0=2, n=0)
    assert m == -math.inf and l == 0.0 and not o.any()
    out, lse = O.merge([m, m], [l, l], [o, o])
    assert lse == -math.inf and not out.any() and not np.isnan(out).any()
    out, lse = O.full(q, K, V, "f16", t0=0, n=0)
    assert lse == -math.inf and not out.any()


def test_partial_from_logits_is_the_hand_off_form_of_partial():
    """Host logits + gathered V rows give the partial of those tokens: against brute force, against PARTIAL
    over an index list, and merged with the device's partial against monolithic attention (the paper's
    workflow: CPU logits for its tokens, GPU logits for its own, one softmax over both)."""
    n, D = 90, 16
    q, K, V = rand_case(n, D, "f16", sigma=1.5)
    out, lse = O.full(q, K, V, "f16")
    host = np.sort(RNG.permutation(n)[:37]); dev = np.setdiff1d(np.arange(n), host)
    s = O.logits(q, K, "f16", idx=host)                                   # what the host's logits calculator sends
    m, l, o = O.partial_from_logits(s, V[host], "f16")
    sd = np_decode(V[host], "f16").astype(np.float64)
    w = np.exp(s - s.max())
    assert m == s.max() and abs(l - w.sum()) < 1e-13
    np.testing.assert_allclose(o, (w[:, None] * sd).sum(axis=0), rtol=0, atol=1e-12)
    pm, pl, po = O.partial(q, K, V, "f16", idx=host)
    assert (m, l) == (pm, pl) and np.array_equal(o, po)
    dm, dl, do = O.partial(q, K, V, "f16", idx=dev)
    mo, ml = O.merge([m, dm], [l, dl], [o, do])
    np.testing.assert_allclose(mo, out, rtol=1e-12, atol=1e-14)
    assert abs(ml - lse) < 1e-12
    lo, ll = O.literal(q, K, V, "f16", host, dev)
    np.testing.assert_allclose(mo, lo, rtol=1e-12, atol=1e-14)
    # unselected slots carry -inf; nothing selected is the empty partial
    s2 = s.copy(); s2[::2] = -np.inf
    m2, l2, o2 = O.partial_from_logits(s2, V[host], "f16")
    m3, l3, o3 = O.partial_from_logits(s[1::2], V[host][1::2], "f16")
    assert (m2, l2) == (m3, l3) and np.array_equal(o2, o3)
    me, le, oe = O.partial_from_logits(np.full(5, -np.inf), V[:5], "f16")
    assert me == -math.inf and le == 0 and not oe.any()


# ---- invariants -------------------------------------------------------------------------------

def test_partial_invariants_and_convex_hull():
    n, D = 64, 8
    q, K, V = rand_case(n, D, "f16")
    s = O.logits(q, K, "f16")
    m, l, o = O.partial(q, K, V, "f16")
    assert m == s.max() and (m >= s).all()
    assert 1.0 <= l <= n
    w = np.exp(s - m) / l
    assert abs(w.sum() - 1.0) < 1e-14
    out, lse = O.full(q, K, V, "f16")
    assert lse >= m
    np.testing.assert_allclose(o / l, out, rtol=1e-13, atol=1e-15)
    Vd = np_decode(V, "f16").astype(np.float64)
    assert (out <= Vd.max(axis=0) + 1e-15).all() and (out >= Vd.min(axis=0) - 1e-15).all()


def test_permutation_and_value_shift_invariance():
    n, D = 50, 8
    q, K, V = rand_case(n, D, "f16")
    out, lse = O.full(q, K, V, "f16")
    p = RNG.permutation(n)
    po, pl = O.full(q, K[p], V[p], "f16")
    np.testing.assert_allclose(po, out, rtol=0, atol=1e-13)
    assert abs(pl - lse) < 1e-13
    # V + c shifts the output by c (c chosen so every sum is exact in fp16)
    Vs = f16_bits(np.round(np_decode(V, "f16").astype(np.float64) * 8) / 8)
    Vc = f16_bits(np.round(np_decode(V, "f16").astype(np.float64) * 8) / 8 + 4.0)
    a, _ = O.full(q, K, Vs, "f16")
    b, _ = O.full(q, K, Vc, "f16")
    np.testing.assert_allclose(b - a, 4.0, rtol=0, atol=1e-13)
    # constant V gives that constant
    c, _ = O.full(q, K, f16_bits(np.full((n, D), -1.25)), "f16")
    np.testing.assert_allclose(c, -1.25, rtol=0, atol=1e-14)


def test_merge_is_associative_and_commutative():
    n, D = 90, 8
    q, K, V = rand_case(n, D, "f16", sigma=2.0)
    P = [O.partial(q, K, V, "f16", t0=a, n=30) for a in (0, 30, 60)]
    m, l, o = [p[0] for p in P], [p[1] for p in P], [p[2] for p in P]
    ref, rl = O.merge(m, l, o)
    r2, l2 = O.merge(m[::-1], l[::-1], o[::-1])
    np.testing.assert_allclose(r2, ref, rtol=1e-13); assert abs(l2 - rl) < 1e-13
    # merge two first; the un-normalised triple (out*L, M, L) is itself a valid partial
    o01, lse01 = O.merge(m[:2], l[:2], o[:2])
    M01 = max(m[:2]); L01 = math.exp(lse01 - M01)
    r3, l3 = O.merge([M01, m[2]], [L01, l[2]], [o01 * L01, o[2]])
    np.testing.assert_allclose(r3, ref, rtol=1e-12); assert abs(l3 - rl) < 1e-12


# ---- closed forms -----------------------------------------------------------------------------

@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_equal_keys_give_mean_of_values(dtype):
    n, D = 37, 8
    q = enc(RNG.standard_normal(D), dtype)
    krow = enc(RNG.standard_normal(D), dtype)
    K = np.tile(krow, (n, 1))
    V = enc(RNG.standard_normal((n, D)), dtype)
    out, lse = O.full(q, K, V, dtype)
    s = float((np_decode(q, dtype) * np_decode(krow, dtype)).sum() / math.sqrt(D))
    np.testing.assert_allclose(out, np_decode(V, dtype).astype(np.float64).mean(axis=0), rtol=0, atol=1e-14)
    assert abs(lse - (s + math.log(n))) < 1e-13
    out0, lse0 = O.full(enc(np.zeros(D), dtype), enc(RNG.standard_normal((n, D)), dtype), V, dtype)
    np.testing.assert_allclose(out0, np_decode(V, dtype).astype(np.float64).mean(axis=0), rtol=0, atol=1e-14)
    assert abs(lse0 - math.log(n)) < 1e-14


def test_dominant_logit_returns_that_value_row():
    n, D = 20, 4
    q = f16_bits([16.0, 0, 0, 0])
    K = f16_bits(np.zeros((n, D))); K[13] = f16_bits([16.0, 0, 0, 0])       # s_13 = 128, others 0
    V = f16_bits(RNG.standard_normal((n, D)))
    out, lse = O.full(q, K, V, "f16")
    Vd = np_decode(V, "f16").astype(np.float64)
    np.testing.assert_allclose(out, Vd[13], rtol=1e-20, atol=1e-40)
    assert lse == 128.0


# ---- hand-worked example (tests/golden/three_logit_example.txt) ----------------------------------

def _golden():
    g = {}
    for line in open(os.path.join(GOLD, "three_logit_example.txt")):
        if line.strip() and not line.startswith("#"):
            k, v = line.split()
            g[k] = float(v)
    return g


def test_hand_worked_three_logit_example():
    g = _golden()
    q = f16_bits([2.0, 0, 0, 0])
    K = f16_bits([[t, 0, 0, 0] for t in range(3)])
    V = f16_bits([[t, 1.0, -t, 10.0 * t] for t in range(3)])
    np.testing.assert_allclose(O.logits(q, K, "f16"), [0.0, 1.0, 2.0], atol=0)
    out, lse = O.full(q, K, V, "f16")
    m, l, o = O.partial(q, K, V, "f16")
    assert m == 2.0 and abs(l - g["l_full"]) < 5e-10 and abs(lse - g["lse_full"]) < 5e-10
    np.testing.assert_allclose(out, [g["out0"], g["out1"], g["out2"], g["out3"]], rtol=0, atol=5e-9)
    a = O.partial(q, K, V, "f16", idx=[0]); b = O.partial(q, K, V, "f16", idx=[1, 2])
    assert a[0] == g["m_a"] and a[1] == g["l_a"] and b[0] == g["m_b"] and abs(b[1] - g["l_b"]) < 5e-10
    mo, ml = O.merge([a[0], b[0]], [a[1], b[1]], [a[2], b[2]])
    assert abs(math.exp(a[0] - b[0]) - g["w_a"]) < 5e-10
    assert abs(math.exp(ml - 2.0) - g["l_merged"]) < 5e-10
    np.testing.assert_allclose(mo, out, rtol=1e-14)
    # softmax weights recovered from a one-hot V
    for t, key in enumerate(("p0", "p1", "p2")):
        onehot = f16_bits([[1.0 if r == t else 0.0, 0, 0, 0] for r in range(3)])
        assert abs(O.full(q, K, onehot, "f16")[0][0] - g[key]) < 5e-10
    _, lse2 = O.full(q, f16_bits([[3, 0, 0, 0], [3, 0, 0, 0]]), V[:2], "f16")
    assert abs(lse2 - (3.0 + g["ln2"])) < 5e-10


# ---- special case that reduces to a library routine ----------------------------------------------

def test_matches_torch_float64_softmax():
    import torch

    n, D = 500, 64
    q, K, V = rand_case(n, D, "f16")
    qd = torch.from_numpy(np_decode(q, "f16").astype(np.float64))
    Kd = torch.from_numpy(np_decode(K, "f16").astype(np.float64))
    Vd = torch.from_numpy(np_decode(V, "f16").astype(np.float64))
    s = (Kd @ qd) / math.sqrt(D)
    ref = torch.softmax(s, dim=0) @ Vd
    out, lse = O.full(q, K, V, "f16")
    np.testing.assert_allclose(out, ref.numpy(), rtol=0, atol=1e-13)
    assert abs(lse - float(torch.logsumexp(s, dim=0))) < 1e-12


# ---- batched forms: head grouping, strides and the chunk grid -----------------------------------

def test_batched_forms_use_consecutive_head_groups_and_absolute_chunk_grid():
    B, Hq, Hkv, D, Lmax = 2, 6, 2, 8, 75
    G = Hq // Hkv
    q = f16_bits(RNG.standard_normal((B, Hq, D)))
    K = f16_bits(RNG.standard_normal((B, Lmax, Hkv, D)))
    V = f16_bits(RNG.standard_normal((B, Lmax, Hkv, D)))
    lo, hi, C = [13, 0], [70, 41], 16
    NC = 5
    m, l, o = O.chunked_partials(q, K, V, "f16", lo, hi, C, NC, threads=3)
    out, lse = O.full_batch(q, K, V, "f16", lo, hi, threads=2)
    for b in range(B):
        first = lo[b] // C
        for h in range(Hq):
            g = h // G                                              # head h reads KV head h div G
            Kr, Vr = np.ascontiguousarray(K[b, :, g]), np.ascontiguousarray(V[b, :, g])
            bo, bl, _ = brute(q[b, h], Kr, Vr, "f16", np.arange(lo[b], hi[b]))
            np.testing.assert_allclose(out[b, h], bo, rtol=0, atol=1e-13)
            assert abs(lse[b, h] - bl) < 1e-13
            for c in range(NC):
                a, e = max((first + c) * C, lo[b]), min((first + c + 1) * C, hi[b])
                pm, pl, po = O.partial(q[b, h], Kr, Vr, "f16", t0=a, n=max(0, e - a))
                assert m[b, h, c] == pm and l[b, h, c] == pl
                np.testing.assert_array_equal(o[b, h, c], po)
            mo, ml = O.merge(m[b, h], l[b, h], o[b, h])
            np.testing.assert_allclose(mo, out[b, h], rtol=1e-12, atol=1e-14)
            assert abs(ml - lse[b, h]) < 1e-12
    mb, lb = O.merge_batch(m, l, o)
    np.testing.assert_allclose(mb, out, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lb, lse, rtol=0, atol=1e-12)


def test_statistical_sanity_of_lse_for_gaussian_keys():
    """Loose check, not a parity pin: for iid keys lse ~ ln n + sigma_s^2 / 2."""
    n, D = 20000, 64
    q, K, V = rand_case(n, D, "f16", sigma=0.5)
    qd = np_decode(q, "f16").astype(np.float64)
    var_s = 0.25 * float((qd ** 2).sum()) / D
    _, lse = O.full(q, K, V, "f16")
    assert abs(lse - (math.log(n) + var_s / 2)) < 0.05

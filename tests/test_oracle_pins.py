"""Pins for the float64 oracle: it is checked against things other than itself.

* exact-rational brute force on tiny inputs (pure Python, `fractions` + `math.fsum`);
* a hand-derived worked example of Eq. 1 (tests/golden/two_token_softmax.txt);
* closed forms and invariants that follow from Eq. 1 (Sec. 2.3) and from composition being a
  concatenation (Sec. 3.1, Sec. 5.4);
* a float64 library softmax-attention on the concatenated cache.
Each is chosen so that a dropped term, a wrong sign, a wrong head index or a transposed operand in
the oracle fails at least one of them.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
from paper_2506_06266_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float values to bf16 (nearest even) and return the bit patterns."""
    t = torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16)
    return synth.bits(t)


def bits_to_fraction(b: int) -> Fraction:
    """Exact value of a finite bf16 bit pattern, decoded field by field."""
    sign = -1 if (b >> 15) & 1 else 1
    e = (b >> 7) & 0xFF
    m = b & 0x7F
    if e == 0:
        return sign * Fraction(m, 1 << 7) * Fraction(1, 1 << 126)
    assert e != 0xFF
    val = Fraction((1 << 7) + m, 1 << 7)
    return sign * (val * (Fraction(2) ** (e - 127)))


def bits_to_float64(b: np.ndarray) -> np.ndarray:
    return (b.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def brute_force(q_bits, segments, scale_frac: Fraction, Hkv: int):
    """Eq. 1 at the last position, one (request, head) at a time, with exact rational scores."""
    B, Hq, D = q_bits.shape
    G = Hq // Hkv
    out = np.zeros((B, Hq, D))
    lse = np.zeros((B, Hq))
    for b in range(B):
        for h in range(Hq):
            g = h // G
            keys, vals = [], []
            for (k, v) in segments[b]:          # the cache, in order: Cartridge(s) then suffix
                for j in range(k.shape[1]):
                    keys.append([bits_to_fraction(int(x)) for x in k[g, j]])
                    vals.append([bits_to_fraction(int(x)) for x in v[g, j]])
            qv = [bits_to_fraction(int(x)) for x in q_bits[b, h]]
            t = [float(scale_frac * sum(a * c for a, c in zip(qv, kj))) for kj in keys]
            M = max(t)
            Z = math.fsum(math.exp(x - M) for x in t)
            lse[b, h] = M + math.log(Z)
            for d in range(D):
                out[b, h, d] = math.fsum(math.exp(x - M) * float(vj[d]) for x, vj in zip(t, vals)) / Z
    return out, lse


def rand_bits(rng, shape, scale=1.0):
    return bf16_bits(rng.standard_normal(shape) * scale)


# ---------------------------------------------------------------------------------------------
def test_bf16_decode_matches_field_decoding():
    # the oracle's bf16 -> double widening, checked through a one-token cache (o = v exactly)
    rng = np.random.default_rng(1)
    v = rng.integers(0, 1 << 16, size=(1, 1, 64), dtype=np.uint16)
    v[(v & 0x7F80) == 0x7F80] = 0x3F80              # no inf / nan
    k = rand_bits(rng, (1, 1, 64))
    q = rand_bits(rng, (1, 1, 64))
    out, _ = oracle.decode_layer(q, [[(k, v)]], 0.125)
    expect = np.array([float(bits_to_fraction(int(x))) for x in v[0, 0]])
    assert np.array_equal(out[0, 0], expect)


@pytest.mark.parametrize("seed,B,Hq,Hkv,D,ps,ss", [
    (11, 2, 4, 2, 4, [1], [0, 2]),
    (12, 2, 4, 2, 4, [3], [2, 1]),
    (13, 3, 6, 2, 4, [3, 1], [2, 0, 5]),      # two composed Cartridges then a suffix
    (14, 1, 3, 1, 16, [], [7]),               # suffix only, MQA-like
    (15, 2, 8, 8, 16, [5], [3, 3]),           # G = 1
])
def test_brute_force_exact_rational(seed, B, Hq, Hkv, D, ps, ss):
    rng = np.random.default_rng(seed)
    q = rand_bits(rng, (B, Hq, D))
    segments = []
    for b in range(B):
        segs = [(rand_bits(rng, (Hkv, p, D)), rand_bits(rng, (Hkv, p, D))) for p in ps]
        if ss[b] > 0:
            segs.append((rand_bits(rng, (Hkv, ss[b], D)), rand_bits(rng, (Hkv, ss[b], D))))
        segments.append(segs)
    root = math.isqrt(D)
    assert root * root == D
    scale = Fraction(1, root)
    out, lse = oracle.decode_layer(q, segments, float(scale))
    bo, bl = brute_force(q, segments, scale, Hkv)
    assert np.max(np.abs(out - bo)) <= 1e-12
    assert np.max(np.abs(lse - bl)) <= 1e-12


def test_golden_two_token_example():
    rows = {"k": [], "v": []}
    with open(os.path.join(GOLDEN, "two_token_softmax.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            key, *vals = line.split()
            vals = [float(x) for x in vals]
            if key in ("k", "v"):
                rows[key].append(vals)
            else:
                rows[key] = vals
    q = bf16_bits(np.array(rows["q"]))[None, None, :]
    k = bf16_bits(np.array(rows["k"]))[None, :, :]
    v = bf16_bits(np.array(rows["v"]))[None, :, :]
    out, lse = oracle.decode_layer(q, [[(k, v)]], rows["scale"][0])
    assert abs(lse[0, 0] - rows["lse"][0]) < 1e-14
    assert np.max(np.abs(out[0, 0] - np.array(rows["o"]))) < 1e-14


def test_one_token_cache_returns_its_value():
    rng = np.random.default_rng(2)
    Hq, Hkv, D = 6, 2, 32
    q = rand_bits(rng, (1, Hq, D))
    k = rand_bits(rng, (Hkv, 1, D))
    v = rand_bits(rng, (Hkv, 1, D))
    out, lse = oracle.decode_layer(q, [[(k, v)]], 0.3)
    G = Hq // Hkv
    qf, kf, vf = bits_to_float64(q), bits_to_float64(k), bits_to_float64(v)
    for h in range(Hq):
        g = h // G
        assert np.array_equal(out[0, h], vf[g, 0])
        assert abs(lse[0, h] - 0.3 * float(qf[0, h] @ kf[g, 0])) < 1e-13


def test_identical_keys_give_mean_of_values():
    rng = np.random.default_rng(3)
    Hq, Hkv, D, n = 4, 2, 16, 37
    q = rand_bits(rng, (1, Hq, D))
    k1 = rand_bits(rng, (Hkv, 1, D))
    k = np.repeat(k1, n, axis=1)
    v = rand_bits(rng, (Hkv, n, D))
    out, lse = oracle.decode_layer(q, [[(k, v)]], 0.25)
    vf, qf, kf = bits_to_float64(v), bits_to_float64(q), bits_to_float64(k1)
    for h in range(Hq):
        g = h // 2
        assert np.max(np.abs(out[0, h] - vf[g].mean(axis=0))) < 1e-13
        assert abs(lse[0, h] - (0.25 * float(qf[0, h] @ kf[g, 0]) + math.log(n))) < 1e-12


def test_zero_query_gives_mean_and_log_n():
    rng = np.random.default_rng(4)
    n = 50
    q = np.zeros((1, 2, 8), dtype=np.uint16)
    k = rand_bits(rng, (1, n, 8))
    v = rand_bits(rng, (1, n, 8))
    out, lse = oracle.decode_layer(q, [[(k, v)]], 1.0)
    assert np.max(np.abs(out[0, 0] - bits_to_float64(v)[0].mean(axis=0))) < 1e-13
    assert np.max(np.abs(lse - math.log(n))) < 1e-13


def test_one_hot_keys_retrieve_the_matching_value():
    # the associative-recall setting of App. E: orthonormal keys, query equal to one of them
    D = 16
    k = bf16_bits(np.eye(D))[None, :, :]
    rng = np.random.default_rng(5)
    v = rand_bits(rng, (1, D, D))
    j = 5
    q = bf16_bits(np.eye(D)[j])[None, None, :]
    out, lse = oracle.decode_layer(q, [[(k, v)]], 200.0)
    assert np.max(np.abs(out[0, 0] - bits_to_float64(v)[0, j])) < 1e-12
    assert abs(lse[0, 0] - 200.0) < 1e-12


def test_key_shift_moves_lse_only():
    rng = np.random.default_rng(6)
    D, n = 8, 20
    # integers keep q, k, c and k + c exact in bf16
    q = bf16_bits(rng.integers(-3, 4, (1, 2, D)))
    kf = rng.integers(-4, 5, (1, n, D)).astype(np.float64)
    c = rng.integers(-2, 3, (D,)).astype(np.float64)
    v = rand_bits(rng, (1, n, D))
    o1, l1 = oracle.decode_layer(q, [[(bf16_bits(kf), v)]], 0.125)
    o2, l2 = oracle.decode_layer(q, [[(bf16_bits(kf + c), v)]], 0.125)
    qf = bits_to_float64(q)
    assert np.max(np.abs(o1 - o2)) < 1e-13
    for h in range(2):
        assert abs((l2[0, h] - l1[0, h]) - 0.125 * float(qf[0, h] @ c)) < 1e-12


def test_duplicated_cache_adds_log2():
    rng = np.random.default_rng(7)
    q = rand_bits(rng, (1, 4, 8))
    k = rand_bits(rng, (2, 9, 8))
    v = rand_bits(rng, (2, 9, 8))
    o1, l1 = oracle.decode_layer(q, [[(k, v)]], 0.5)
    o2, l2 = oracle.decode_layer(q, [[(k, v), (k, v)]], 0.5)
    assert np.max(np.abs(o1 - o2)) < 1e-13
    assert np.max(np.abs(l2 - l1 - math.log(2))) < 1e-13


def test_concatenation_equals_lse_merge_of_parts():
    rng = np.random.default_rng(8)
    Hq, Hkv, D = 6, 2, 16
    q = rand_bits(rng, (2, Hq, D))
    A = (rand_bits(rng, (Hkv, 13, D)), rand_bits(rng, (Hkv, 13, D)))
    Bp = (rand_bits(rng, (Hkv, 5, D)), rand_bits(rng, (Hkv, 5, D)))
    S = (rand_bits(rng, (Hkv, 3, D)), rand_bits(rng, (Hkv, 3, D)))
    full, lfull = oracle.decode_layer(q, [[A, Bp, S], [A, Bp, S]], 0.25)
    parts = [oracle.decode_layer(q, [[x], [x]], 0.25) for x in (A, Bp, S)]
    lses = np.stack([p[1] for p in parts])                       # [3][B][Hq]
    M = lses.max(axis=0)
    tot = M + np.log(np.exp(lses - M).sum(axis=0))
    merged = sum(np.exp(p[1] - tot)[..., None] * p[0] for p in parts)
    assert np.max(np.abs(tot - lfull)) < 1e-12
    assert np.max(np.abs(merged - full)) < 1e-12


def test_compose_equals_single_cartridge_holding_concatenation():
    rng = np.random.default_rng(9)
    L, Hq, Hkv, D = 2, 4, 2, 8
    oc = oracle.OracleCache(L, Hq, Hkv, D, 0.35)
    ka, va = rand_bits(rng, (L, Hkv, 6, D)), rand_bits(rng, (L, Hkv, 6, D))
    kb, vb = rand_bits(rng, (L, Hkv, 4, D)), rand_bits(rng, (L, Hkv, 4, D))
    a, b = oc.register(ka, va), oc.register(kb, vb)
    ab = oc.compose([a, b])
    cat = oc.register(np.concatenate([ka, kb], axis=2), np.concatenate([va, vb], axis=2))
    ba = oc.compose([b, a])
    r1, r2, r3 = oc.open(ab), oc.open(cat), oc.open(ba)
    ks, vs = rand_bits(rng, (3, Hkv, D)), rand_bits(rng, (3, Hkv, D))
    for layer in range(L):
        # every request appends the same suffix token
        oc.append(layer, [r1, r2, r3], np.repeat(ks[:1], 3, 0), np.repeat(vs[:1], 3, 0))
    q = rand_bits(rng, (1, Hq, D))
    q3 = np.repeat(q, 3, axis=0)
    for layer in range(L):
        out, lse = oc.decode(layer, [r1, r2, r3], q3)
        assert np.array_equal(out[0], out[1]) and np.array_equal(lse[0], lse[1])
        # keys are stored post-RoPE, so the order of the parts only changes rounding
        assert np.max(np.abs(out[0] - out[2])) < 1e-13
        assert np.max(np.abs(lse[0] - lse[2])) < 1e-13
    assert oc.kv_tokens(0, r1) == 11


def test_permuting_cache_rows_changes_nothing_but_rounding():
    rng = np.random.default_rng(10)
    q = rand_bits(rng, (1, 4, 16))
    k = rand_bits(rng, (2, 31, 16))
    v = rand_bits(rng, (2, 31, 16))
    perm = rng.permutation(31)
    o1, l1 = oracle.decode_layer(q, [[(k, v)]], 0.25)
    o2, l2 = oracle.decode_layer(q, [[(k[:, perm], v[:, perm])]], 0.25)
    assert np.max(np.abs(o1 - o2)) < 1e-13 and np.max(np.abs(l1 - l2)) < 1e-13


def test_output_is_a_convex_combination_of_values():
    rng = np.random.default_rng(16)
    q = rand_bits(rng, (2, 4, 8), 3.0)
    segs = [[(rand_bits(rng, (2, 12, 8)), rand_bits(rng, (2, 12, 8)))] for _ in range(2)]
    out, _ = oracle.decode_layer(q, segs, 0.7)
    for b in range(2):
        vf = bits_to_float64(segs[b][0][1])
        for h in range(4):
            g = h // 2
            assert np.all(out[b, h] <= vf[g].max(axis=0) + 1e-12)
            assert np.all(out[b, h] >= vf[g].min(axis=0) - 1e-12)


def test_gqa_heads_of_a_group_share_kv_and_groups_do_not():
    rng = np.random.default_rng(17)
    Hq, Hkv, D = 6, 2, 8
    q = rand_bits(rng, (1, Hq, D))
    k = rand_bits(rng, (Hkv, 9, D))
    v = rand_bits(rng, (Hkv, 9, D))
    out, lse = oracle.decode_layer(q, [[(k, v)]], 0.4)
    # swapping two query heads inside a group permutes the outputs
    q2 = q.copy()
    q2[0, [0, 2]] = q[0, [2, 0]]
    out2, lse2 = oracle.decode_layer(q2, [[(k, v)]], 0.4)
    assert np.array_equal(out2[0, 0], out[0, 2]) and np.array_equal(out2[0, 2], out[0, 0])
    assert lse2[0, 0] == lse[0, 2]
    # the same query in heads of different groups sees different K/V: contiguous grouping g = h // G
    q3 = np.repeat(q[:, :1], Hq, axis=1)
    out3, _ = oracle.decode_layer(q3, [[(k, v)]], 0.4)
    assert np.array_equal(out3[0, 0], out3[0, 1]) and np.array_equal(out3[0, 1], out3[0, 2])
    assert np.array_equal(out3[0, 3], out3[0, 5])
    assert not np.allclose(out3[0, 2], out3[0, 3])


@pytest.mark.parametrize("seed", [21, 22])
def test_matches_library_softmax_attention_float64(seed):
    rng = np.random.default_rng(seed)
    B, Hq, Hkv, D = 3, 12, 4, 128
    G = Hq // Hkv
    q = rand_bits(rng, (B, Hq, D))
    segments, ref_o, ref_l = [], [], []
    for b in range(B):
        lens = [int(rng.integers(1, 200)), int(rng.integers(1, 70))]
        segs = [(rand_bits(rng, (Hkv, n, D)), rand_bits(rng, (Hkv, n, D))) for n in lens]
        segments.append(segs)
        K = np.concatenate([bits_to_float64(s[0]) for s in segs], axis=1)   # [Hkv][n][D]
        V = np.concatenate([bits_to_float64(s[1]) for s in segs], axis=1)
        Kt = torch.from_numpy(np.repeat(K, G, axis=0))[None]                # [1][Hq][n][D]
        Vt = torch.from_numpy(np.repeat(V, G, axis=0))[None]
        Qt = torch.from_numpy(bits_to_float64(q[b]))[None, :, None, :]      # [1][Hq][1][D]
        o = torch.nn.functional.scaled_dot_product_attention(Qt, Kt, Vt, scale=D ** -0.5)
        ref_o.append(o[0, :, 0].numpy())
        s = (Qt @ Kt.transpose(-1, -2))[0, :, 0] * D ** -0.5
        ref_l.append(torch.logsumexp(s, dim=-1).numpy())
    out, lse = oracle.decode_layer(q, segments, D ** -0.5)
    assert np.max(np.abs(out - np.stack(ref_o))) < 1e-12
    assert np.max(np.abs(lse - np.stack(ref_l))) < 1e-12


def test_empty_cache_is_rejected_and_empty_parts_are_allowed():
    rng = np.random.default_rng(23)
    q = rand_bits(rng, (1, 2, 8))
    empty = (np.zeros((1, 0, 8), np.uint16), np.zeros((1, 0, 8), np.uint16))
    seg = (rand_bits(rng, (1, 4, 8)), rand_bits(rng, (1, 4, 8)))
    with pytest.raises(ValueError):
        oracle.decode_layer(q, [[empty]], 1.0)
    o1, l1 = oracle.decode_layer(q, [[seg]], 1.0)
    o2, l2 = oracle.decode_layer(q, [[empty, seg, empty]], 1.0)
    assert np.array_equal(o1, o2) and np.array_equal(l1, l2)


def test_append_and_extend_grow_the_suffix_in_order():
    rng = np.random.default_rng(24)
    L, Hq, Hkv, D = 1, 2, 2, 8
    oc = oracle.OracleCache(L, Hq, Hkv, D, 0.5)
    r = oc.open(None)
    toks_k = rand_bits(rng, (5, Hkv, D))
    toks_v = rand_bits(rng, (5, Hkv, D))
    oc.extend(0, r, toks_k[:3], toks_v[:3])
    oc.append(0, [r], toks_k[3:4], toks_v[3:4])
    oc.append(0, [r], toks_k[4:5], toks_v[4:5])
    assert oc.suffix_len(r, 0) == 5
    (k, v), = oc.segments(0, r)
    assert np.array_equal(k, np.transpose(toks_k, (1, 0, 2)))
    assert np.array_equal(v, np.transpose(toks_v, (1, 0, 2)))


def test_cartridge_footprint_matches_printed_sizes():
    w = synth.config3()
    per_token_layer = w.kv_bytes_per_token_layer()
    assert per_token_layer == 4096
    with open(os.path.join(GOLDEN, "cartridge_footprint.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            layers, p, gb, tol = line.split()
            size = int(layers) * int(p) * per_token_layer / 1e9
            assert abs(size - float(gb)) <= float(tol)

"""Pins for the FP8 (e4m3) oracle: the codec against the format's definition and an independent library
conversion, whole-page quantisation against its defining properties, FP8 attention against the already
pinned bf16 oracle on inputs where both must agree exactly, the one-token append against separately written
index arithmetic. CPU only."""
import math

import numpy as np
import pytest
import torch

import oracle

P = 16


def bits(x):
    return oracle.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


# ---------------------------------------------------------------- codec

def test_e4m3_decode_matches_the_format_definition_and_torch():
    codes = np.arange(256, dtype=np.uint8)
    got = oracle.e4m3_to_f64(codes)
    # the format's own values (tests/golden/e4m3_codes.txt: bias 7, subnormals m/8 * 2^-6, S.1111.111 is NaN)
    import os

    n_checked = 0
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "e4m3_codes.txt")):
        if line.startswith("#") or not line.strip():
            continue
        code, value = line.split()
        c, v = int(code, 16), float(value)
        if math.isnan(v):
            assert math.isnan(got[c])
        else:
            assert got[c] == v and math.copysign(1.0, got[c]) == math.copysign(1.0, v)
        n_checked += 1
    assert n_checked == 19
    ref = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    finite = ~np.isnan(ref)
    assert finite.sum() == 254 and np.array_equal(got[finite], ref[finite])
    # strictly increasing over the positive finite codes
    assert np.all(np.diff(got[:0x7F]) > 0)


def test_e4m3_encode_round_trips_rounds_to_even_and_saturates():
    codes = np.array([c for c in range(256) if c & 0x7F != 0x7F], dtype=np.uint8)
    vals = oracle.e4m3_to_f64(codes).astype(np.float32)
    back = oracle.f32_to_e4m3(vals)
    assert np.array_equal(back[codes != 0x80], codes[codes != 0x80])  # -0 keeps its sign bit too
    assert back[list(codes).index(0x80)] == 0x80
    # ties go to the even mantissa: 1.0625 is halfway between 1.0 (m=0) and 1.125 (m=1)
    assert list(oracle.f32_to_e4m3([1.0625, 1.1875, 1.3125, 2.0 ** -10, 3 * 2.0 ** -10])) == [0x38, 0x3A, 0x3A, 0x00, 0x02]
    assert list(oracle.f32_to_e4m3([448.0, 449.0, 463.9, 464.0, 1e30, np.inf, -1e30])) == [0x7E] * 6 + [0xFE]
    assert oracle.f32_to_e4m3([np.nan])[0] == 0x7F
    # every midpoint between neighbours, nudged down and up, lands on the lower and the upper neighbour
    pos = oracle.e4m3_to_f64(np.arange(0x7F, dtype=np.uint8))
    mid = (pos[:-1] + pos[1:]) / 2
    lo = oracle.f32_to_e4m3(np.nextafter(mid.astype(np.float32), np.float32(0)))
    hi = oracle.f32_to_e4m3(np.nextafter(mid.astype(np.float32), np.float32(1e9)))
    assert np.array_equal(lo, np.arange(0x7E)) and np.array_equal(hi, np.arange(1, 0x7F))


def test_e4m3_encode_matches_torch_inside_the_finite_range():
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * 3, rng.uniform(-448, 448, 20000),
                        rng.standard_normal(5000) * 1e-2, rng.standard_normal(5000) * 1e-3]).astype(np.float32)
    ref = torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()
    got = oracle.f32_to_e4m3(x)
    assert np.array_equal(got, ref)


# ---------------------------------------------------------------- whole-page quantisation

def test_quantize_pages_scale_codes_and_error_bound():
    rng = np.random.default_rng(1)
    NP, Hkv, d = 5, 2, 64
    k = bits(rng.standard_normal((NP, Hkv, P, d)) * 3)
    v = bits(rng.standard_normal((NP, Hkv, P, d)) * 0.1)
    tip = np.array([16, 16, 5, 0, 1], dtype=np.int32)
    k[2, :, 5:] = 0x7FC0  # NaN poison in the slots that hold no token
    k[3] = 0x7FC0
    k8, v8, sc = oracle.fp8_quantize_pages(k, v, tip)
    kf = oracle.bf16_bits_to_f64(k)
    for p in range(NP):
        for h in range(Hkv):
            n = tip[p]
            assert np.all(k8[p, h, n:] == 0) and np.all(v8[p, h, n:] == 0)
            if n == 0:
                assert sc[p, h, 0] == 1.0 and sc[p, h, 1] == 1.0
                continue
            amax = np.abs(kf[p, h, :n]).max()
            assert sc[p, h, 0] == np.float32(np.float32(amax) / np.float32(448.0))
            assert sc[p, h, 2] == 0 and sc[p, h, 3] == 0
            deq = float(sc[p, h, 0]) * oracle.e4m3_to_f64(k8[p, h, :n])
            # the largest element lands on +-448; every element is within half a code step of its value
            assert np.abs(oracle.e4m3_to_f64(k8[p, h, :n])).max() == 448.0
            step = np.maximum(2.0 ** (np.floor(np.log2(np.maximum(np.abs(kf[p, h, :n]) / float(sc[p, h, 0]), 2.0 ** -6))) - 3), 2.0 ** -9)
            assert np.all(np.abs(deq - kf[p, h, :n]) <= 0.5 * step * float(sc[p, h, 0]) * (1 + 1e-6))


# ---------------------------------------------------------------- attention over FP8 pages

def small_fp8_cache(rng, lens, Hkv, d, pow2_scales):
    n_pages = int(sum((L + P - 1) // P for L in lens)) + 2
    perm = rng.permutation(n_pages).astype(np.int32)
    MP = max(1, max((L + P - 1) // P for L in lens))
    table = np.full((len(lens), MP), -1, dtype=np.int32)
    cur = 0
    for b, L in enumerate(lens):
        n = (L + P - 1) // P
        table[b, :n] = perm[cur:cur + n]
        cur += n
    k8 = rng.integers(0, 256, size=(n_pages, Hkv, P, d)).astype(np.uint8)
    v8 = rng.integers(0, 256, size=(n_pages, Hkv, P, d)).astype(np.uint8)
    k8[(k8 & 0x7F) == 0x7F] = 0x38  # no NaN codes inside contexts
    v8[(v8 & 0x7F) == 0x7F] = 0xB8
    k8[(k8 & 0x7F) > 0x50] &= 0xCF  # keep logits moderate
    sc = np.zeros((n_pages, Hkv, 4), dtype=np.float32)
    if pow2_scales:
        sc[..., 0] = 2.0 ** rng.integers(-6, -2, size=(n_pages, Hkv))
        sc[..., 1] = 2.0 ** rng.integers(-4, 3, size=(n_pages, Hkv))
    else:
        sc[..., 0] = rng.uniform(0.01, 0.1, size=(n_pages, Hkv))
        sc[..., 1] = rng.uniform(0.05, 2.0, size=(n_pages, Hkv))
    return k8, v8, sc, table


@pytest.mark.parametrize("g,d", [(1, 64), (4, 64), (8, 128)])
def test_fp8_attention_equals_the_bf16_oracle_when_dequantisation_is_exact(g, d):
    """e4m3 has 4 significant bits and the scales here are powers of two, so scale * code is a bf16 value:
    the pinned bf16 oracle on the dequantised cache must give the same result."""
    rng = np.random.default_rng(10 + g)
    lens = [1, 15, 16, 17, 40, 0, 100]
    Hkv = 2
    k8, v8, sc, table = small_fp8_cache(rng, lens, Hkv, d, pow2_scales=True)
    kd = sc[..., 0][:, :, None, None].astype(np.float64) * oracle.e4m3_to_f64(k8)
    vd = sc[..., 1][:, :, None, None].astype(np.float64) * oracle.e4m3_to_f64(v8)
    kb, vb = bits(kd), bits(vd)
    assert np.array_equal(oracle.bf16_bits_to_f64(kb), kd) and np.array_equal(oracle.bf16_bits_to_f64(vb), vd)
    q = bits(rng.standard_normal((len(lens), g * Hkv, d)))
    lens = np.array(lens, dtype=np.int32)
    out8, lse8 = oracle.fp8_decode_attn(q, k8, v8, sc, table, lens, 0.125)
    out, lse = oracle.decode_attn(q, kb, vb, table, lens, 0.125)
    assert np.allclose(out8, out, rtol=1e-12, atol=1e-13)
    assert np.array_equal(np.isneginf(lse8), np.isneginf(lse))
    ok = ~np.isneginf(lse)
    assert np.allclose(lse8[ok], lse[ok], rtol=1e-12, atol=1e-12)
    assert np.all(out8[lens == 0] == 0)


def test_fp8_attention_brute_force_with_arbitrary_scales():
    rng = np.random.default_rng(20)
    lens = [3, 18]
    Hkv, g, d = 2, 2, 64
    k8, v8, sc, table = small_fp8_cache(rng, lens, Hkv, d, pow2_scales=False)
    q = bits(rng.standard_normal((2, g * Hkv, d)))
    out8, lse8 = oracle.fp8_decode_attn(q, k8, v8, sc, table, np.array(lens, dtype=np.int32), 0.2, nthreads=1)
    qf = oracle.bf16_bits_to_f64(q)
    scale = float(np.float32(0.2))
    for b, L in enumerate(lens):
        for h in range(g * Hkv):
            kvh = h // g
            s, vals = [], []
            for t in range(L):
                page = table[b, t // P]
                kt = float(sc[page, kvh, 0]) * oracle.e4m3_to_f64(k8[page, kvh, t % P])
                vals.append(float(sc[page, kvh, 1]) * oracle.e4m3_to_f64(v8[page, kvh, t % P]))
                s.append(scale * sum(float(a) * float(c) for a, c in zip(qf[b, h], kt)))
            m = max(s)
            w = [math.exp(x - m) for x in s]
            Z = sum(w)
            ref = sum(wi * vi for wi, vi in zip(w, vals)) / Z
            assert np.allclose(out8[b, h], ref, rtol=1e-11, atol=1e-12)
            assert abs(lse8[b, h] - (m + math.log(Z))) < 1e-11


# ---------------------------------------------------------------- one-token append

def test_fp8_append_against_separate_index_arithmetic():
    rng = np.random.default_rng(30)
    Hkv, d, NP, MP = 2, 64, 9, 3
    lens = np.array([0, 5, 16, 31, 48, -1], dtype=np.int32)  # opens a page, inside, opens, fills, no room, invalid
    table = np.array([[0, 1, 2], [3, -1, -1], [4, 5, -1], [6, 7, -1], [8, 8, 8], [0, 0, 0]], dtype=np.int32)
    table[3, 1] = 99  # bad page id at the append position of sequence 3
    k8 = rng.integers(0, 127, size=(NP, Hkv, P, d)).astype(np.uint8)
    v8 = rng.integers(0, 127, size=(NP, Hkv, P, d)).astype(np.uint8)
    sc = np.zeros((NP, Hkv, 4), dtype=np.float32)
    sc[..., 0] = rng.uniform(0.005, 0.02, size=(NP, Hkv))
    sc[..., 1] = rng.uniform(0.001, 0.004, size=(NP, Hkv))  # small: some V elements will saturate
    kn = rng.standard_normal((6, Hkv, d)).astype(np.float32)
    vn = rng.standard_normal((6, Hkv, d)).astype(np.float32)
    knb, vnb = bits(kn), bits(vn)
    knf, vnf = oracle.bf16_bits_to_f64(knb).astype(np.float32), oracle.bf16_bits_to_f64(vnb).astype(np.float32)
    want_k, want_v, want_sc, want_lens = k8.copy(), v8.copy(), sc.copy(), lens.copy()

    def cast(x):  # torch's conversion for values inside the finite range, explicit saturation outside
        x = np.clip(x, -448.0, 448.0).astype(np.float32)
        return torch.from_numpy(x).to(torch.float8_e4m3fn).view(torch.uint8).numpy()

    for b in (0, 1, 2):  # the sequences that can be appended
        pos = int(lens[b])
        page, slot = table[b, pos // P], pos % P
        for h in range(Hkv):
            for which, (src, dst) in enumerate(((knf, want_k), (vnf, want_v))):
                if slot == 0:
                    want_sc[page, h, which] = np.float32(np.abs(src[b, h]).max() * np.float32(2.0)) / np.float32(448.0)
                dst[page, h, slot] = cast(src[b, h] / want_sc[page, h, which])
        want_lens[b] = pos + 1
    n = oracle.fp8_kv_append(knb, vnb, k8, v8, sc, table, lens)
    assert n == 3
    assert np.array_equal(lens, want_lens)
    assert np.array_equal(sc, want_sc)
    assert np.array_equal(k8, want_k) and np.array_equal(v8, want_v)
    # the stored-scale path really saturated somewhere, and a fresh page keeps a factor two of headroom
    assert (np.abs(oracle.e4m3_to_f64(v8[3, :, 5])) == 448.0).any()
    assert np.abs(oracle.e4m3_to_f64(k8[0, :, 0])).max() == 224.0


# ---------------------------------------------------------------- page gather / scatter

def test_fp8_gather_layout_and_scatter_round_trip():
    rng = np.random.default_rng(40)
    NP, Hkv, d = 11, 2, 64
    k8 = rng.integers(0, 256, size=(NP, Hkv, P, d)).astype(np.uint8)
    v8 = rng.integers(0, 256, size=(NP, Hkv, P, d)).astype(np.uint8)
    sc = rng.uniform(0.01, 2.0, size=(NP, Hkv, 4)).astype(np.float32)
    table = np.array([[3, 7, 1, -1], [10, 0, 5, 2]], dtype=np.int32)
    pb, pe = np.array([1, 0]), np.array([3, 4])
    off = np.array([4, 0])  # sequence 1's pages first, then sequence 0's
    packed = oracle.fp8_kv_gather(k8, v8, sc, table, pb, pe, off, 6)
    block = Hkv * P * d
    assert packed.shape == (6, 2 * block + Hkv * 16)
    # packed page 4 is logical page 1 of sequence 0 = pool page 7; packed page 2 is pool page 5
    for row, page in ((4, 7), (5, 1), (0, 10), (1, 0), (2, 5), (3, 2)):
        assert packed[row, :block].tobytes() == k8[page].tobytes()
        assert packed[row, block:2 * block].tobytes() == v8[page].tobytes()
        assert packed[row, 2 * block:].tobytes() == sc[page].tobytes()
    # scatter into a differently numbered destination and read the same logical pages back
    dst_table = np.array([[9, 8, 7, 6], [5, 4, 3, 2]], dtype=np.int32)
    dk, dv, ds = np.zeros_like(k8), np.zeros_like(v8), np.zeros_like(sc)
    oracle.fp8_kv_scatter(packed, off, dk, dv, ds, dst_table, pb, pe)
    for b in range(2):
        for lp in range(pb[b], pe[b]):
            s, t = table[b, lp], dst_table[b, lp]
            assert np.array_equal(dk[t], k8[s]) and np.array_equal(dv[t], v8[s]) and np.array_equal(ds[t], sc[s])
    untouched = sorted(set(range(NP)) - {8, 7, 5, 4, 3, 2})
    assert not dk[untouched].any() and not ds[untouched].any()

"""Pins for the CPU oracle: closed forms, invariants, brute force, a second formulation.

None of these tests touches a GPU or the CUDA library. Each is chosen so that a
plausible mistake in the oracle (dropped scale, wrong head grouping, wrong page
index, transposed operand, reading a masked slot, unstable softmax) fails it.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import oracle
import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "closed_forms.txt")


def golden():
    vals = {}
    with open(GOLDEN) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                vals[k] = float(v)
    return vals


def bf16(x) -> np.ndarray:
    """fp values -> bf16 bit patterns (values used here are bf16-exact or rounded RNE)."""
    return oracle.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))


def tiny_cache(K, V, P=16, perm_seed=0, pool_extra=3):
    """K, V: float arrays [L, Hkv, d] for ONE sequence -> paged pools with permuted pages."""
    L, Hkv, d = K.shape
    npg = max(1, (L + P - 1) // P)
    NP = npg + pool_extra
    rng = np.random.default_rng(perm_seed)
    phys = rng.permutation(NP)[:npg].astype(np.int32)
    kp = np.full((NP, Hkv, P, d), wl.NAN_BF16_BITS, dtype=np.uint16)
    vp = np.full((NP, Hkv, P, d), wl.NAN_BF16_BITS, dtype=np.uint16)
    kb, vb = bf16(K), bf16(V)
    for t in range(L):
        kp[phys[t // P], :, t % P, :] = kb[t]
        vp[phys[t // P], :, t % P, :] = vb[t]
    table = np.full((1, npg + 2), -1, dtype=np.int32)
    table[0, :npg] = phys
    return kp, vp, table, np.array([L], dtype=np.int32)


def rand_case(seed, L, Hq, Hkv, d):
    rng = np.random.default_rng(seed)
    q = rng.standard_normal((1, Hq, d)).astype(np.float32)
    K = rng.standard_normal((L, Hkv, d)).astype(np.float32)
    V = rng.standard_normal((L, Hkv, d)).astype(np.float32)
    return q, K, V


# ---------------------------------------------------------------- closed forms

def test_one_token_context_returns_that_v_exactly():
    q, K, V = rand_case(1, 1, 8, 2, 64)
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    vb = oracle.bf16_bits_to_f64(bf16(V))  # [1, Hkv, d]
    for h in range(8):
        assert np.array_equal(out[0, h], vb[0, h // 4])
        s0 = 0.125 * np.dot(oracle.bf16_bits_to_f64(bf16(q))[0, h], oracle.bf16_bits_to_f64(bf16(K))[0, h // 4])
        assert lse[0, h] == pytest.approx(s0, rel=1e-14, abs=1e-14)


def test_identical_keys_give_mean_of_v():
    rng = np.random.default_rng(2)
    L, Hq, Hkv, d = 37, 4, 2, 64
    q = rng.standard_normal((1, Hq, d)).astype(np.float32)
    k0 = rng.standard_normal((1, Hkv, d)).astype(np.float32)
    K = np.repeat(k0, L, axis=0)
    V = rng.standard_normal((L, Hkv, d)).astype(np.float32)
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    vb = oracle.bf16_bits_to_f64(bf16(V))
    qb, kb = oracle.bf16_bits_to_f64(bf16(q)), oracle.bf16_bits_to_f64(bf16(k0))
    for h in range(Hq):
        np.testing.assert_allclose(out[0, h], vb[:, h // 2].mean(axis=0), rtol=1e-13, atol=1e-15)
        s = 0.125 * np.dot(qb[0, h], kb[0, h // 2])
        assert lse[0, h] == pytest.approx(s + math.log(L), rel=1e-13)


def test_closed_form_two_tokens_tanh_half():
    g = golden()
    d = 64
    q = np.zeros((1, 1, d), np.float32); q[0, 0, 0] = 8.0
    K = np.zeros((2, 1, d), np.float32); K[0, 0, 0] = 1.0
    V = np.stack([np.ones((1, d), np.float32), -np.ones((1, d), np.float32)])
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    assert g["two_tokens.out"] == pytest.approx(math.tanh(0.5), rel=1e-15)
    np.testing.assert_allclose(out[0, 0], g["two_tokens.out"], rtol=1e-14)
    assert lse[0, 0] == pytest.approx(g["two_tokens.lse"], rel=1e-14)
    assert lse[0, 0] == pytest.approx(math.log1p(math.e), rel=1e-14)


def test_closed_form_three_tokens_unit_vectors():
    g = golden()
    d = 64
    q = np.zeros((1, 1, d), np.float32); q[0, 0, 0] = 8.0
    K = np.zeros((3, 1, d), np.float32); K[0, 0, 0] = 1.0; K[1, 0, 0] = 2.0
    V = np.zeros((3, 1, d), np.float32)
    for t in range(3):
        V[t, 0, t] = 1.0
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    Z = 1.0 + math.e + math.e ** 2
    expect = [math.e / Z, math.e ** 2 / Z, 1.0 / Z]
    for t in range(3):
        assert out[0, 0, t] == pytest.approx(g[f"three_tokens.out{t}"], rel=1e-14)
        assert out[0, 0, t] == pytest.approx(expect[t], rel=1e-14)
    assert np.all(out[0, 0, 3:] == 0.0)
    assert lse[0, 0] == pytest.approx(g["three_tokens.lse"], rel=1e-14)
    # the same context split as {0} and {1,2}, merged by LSE, gives the same numbers
    o_a, l_a = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125, t_begin=[0], t_end=[1])
    o_b, l_b = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125, t_begin=[1], t_end=[3])
    om, lm = oracle.lse_merge(np.stack([o_a[0, 0], o_b[0, 0]]), np.array([l_a[0, 0], l_b[0, 0]]))
    np.testing.assert_allclose(om, out[0, 0], rtol=1e-14, atol=1e-16)
    assert lm == pytest.approx(g["three_tokens.lse"], rel=1e-14)


def test_scale_is_applied_to_logits_not_outputs():
    # doubling sm_scale must act like doubling q (exact in bf16), not like scaling V
    q, K, V = rand_case(3, 23, 2, 1, 64)
    kp, vp, table, lens = tiny_cache(K, V)
    o1, l1 = oracle.decode_attn(bf16(2 * oracle.bf16_bits_to_f64(bf16(q))), kp, vp, table, lens, 0.125)
    o2, l2 = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.25)
    np.testing.assert_allclose(o1, o2, rtol=1e-13)
    np.testing.assert_allclose(l1, l2, rtol=1e-13)


# ---------------------------------------------------------------- brute force / second formulation

def brute_force_row(qf, Kf, Vf, scale):
    """Third formulation: pure-Python loops over plain lists (tiny inputs only)."""
    L, d = len(Kf), len(qf)
    s = []
    for t in range(L):
        acc = 0.0
        for j in range(d):
            acc += qf[j] * Kf[t][j]
        s.append(scale * acc)
    m = max(s)
    w = [math.exp(x - m) for x in s]
    Z = math.fsum(w)
    out = [math.fsum(w[t] * Vf[t][j] for t in range(L)) / Z for j in range(d)]
    return out, m + math.log(Z)


@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (4, 1), (8, 2)])
def test_brute_force_tiny(Hq, Hkv):
    d = 64
    g = Hq // Hkv
    rng = np.random.default_rng(10 + Hq)
    B = 3
    lens = np.array([1, 17, 40], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=5, poison=True)
    q = wl.random_bf16((B, Hq, d), 77)
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    out, lse = oracle.decode_attn(oracle.bf16_bits(q), kp, vp, cache.page_table_host, lens, 0.125)
    kf, vf, qf = oracle.bf16_bits_to_f64(kp), oracle.bf16_bits_to_f64(vp), q.double().numpy()
    for b in range(B):
        for h in range(Hq):
            Kl = [kf[cache.page_table_host[b, t // 16], h // g, t % 16].tolist() for t in range(lens[b])]
            Vl = [vf[cache.page_table_host[b, t // 16], h // g, t % 16].tolist() for t in range(lens[b])]
            o, l = brute_force_row(qf[b, h].tolist(), Kl, Vl, 0.125)
            np.testing.assert_allclose(out[b, h], o, rtol=1e-12, atol=1e-14)
            assert lse[b, h] == pytest.approx(l, rel=1e-12)
    assert rng is not None


def numpy_formulation(q_bits, kp, vp, table, lens, scale, Hq):
    """Second formulation, written separately: gather the whole context with fancy
    indexing, build the explicit probability vector in long double, one mat-vec."""
    B = len(lens)
    NP, Hkv, P, d = kp.shape
    g = Hq // Hkv
    out = np.zeros((B, Hq, d))
    lse = np.zeros((B, Hq))
    qf = oracle.bf16_bits_to_f64(q_bits).astype(np.longdouble)
    for b in range(B):
        L = int(lens[b])
        t = np.arange(L)
        pages = table[b, t // P]
        for h in range(Hq):
            Kc = oracle.bf16_bits_to_f64(kp[pages, h // g, t % P]).astype(np.longdouble)  # [L, d]
            Vc = oracle.bf16_bits_to_f64(vp[pages, h // g, t % P]).astype(np.longdouble)
            s = np.longdouble(np.float32(scale)) * (Kc @ qf[b, h])
            lz = np.log(np.sum(np.exp(s - s.max()))) + s.max()
            p = np.exp(s - lz)
            out[b, h] = (p @ Vc).astype(np.float64)
            lse[b, h] = float(lz)
    return out, lse


@pytest.mark.parametrize("Hq,Hkv,d,maxlen", [(8, 2, 64, 300), (32, 8, 128, 700), (8, 1, 128, 4096), (2, 2, 64, 100)])
def test_independent_numpy_formulation(Hq, Hkv, d, maxlen):
    rng = np.random.default_rng(Hq * 131 + d)
    B = 3
    lens = rng.integers(1, maxlen, size=B, endpoint=True).astype(np.int32)
    lens[0] = maxlen
    cache = wl.build_paged_cache(lens, Hkv, d, seed=Hq + d, poison=True)
    q = oracle.bf16_bits(wl.random_bf16((B, Hq, d), 4242))
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    scale = 1.0 / math.sqrt(d)
    out, lse = oracle.decode_attn(q, kp, vp, cache.page_table_host, lens, scale)
    o2, l2 = numpy_formulation(q, kp, vp, cache.page_table_host, lens, scale, Hq)
    np.testing.assert_allclose(out, o2, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lse, l2, rtol=1e-12, atol=1e-13)
    assert np.all(np.isfinite(out))


def test_matches_torch_sdpa_on_dense_layout():
    """A library routine on the special case it covers: contiguous pages, g = 1."""
    d, L, H = 64, 48, 2
    q, K, V = rand_case(8, L, H, H, d)
    kp, vp, table, lens = tiny_cache(K, V, perm_seed=3)
    out, _ = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    qt = torch.from_numpy(oracle.bf16_bits_to_f64(bf16(q))).permute(1, 0, 2)[None]  # [1,H,1,d]
    kt = torch.from_numpy(oracle.bf16_bits_to_f64(bf16(K))).permute(1, 0, 2)[None]  # [1,H,L,d]
    vt = torch.from_numpy(oracle.bf16_bits_to_f64(bf16(V))).permute(1, 0, 2)[None]
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, scale=0.125)[0, :, 0].numpy()
    np.testing.assert_allclose(out[0], ref, rtol=1e-12, atol=1e-14)


# ---------------------------------------------------------------- invariants

def test_gqa_mapping_is_contiguous_groups():
    Hq, Hkv, d, L = 8, 2, 64, 29
    rng = np.random.default_rng(6)
    q = rng.standard_normal((1, Hq, d)).astype(np.float32)
    K = rng.standard_normal((L, Hkv, d)).astype(np.float32)
    V = np.empty((L, Hkv, d), np.float32)
    for kvh in range(Hkv):
        V[:, kvh, :] = kvh + 1
    kp, vp, table, lens = tiny_cache(K, V)
    out, _ = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    for h in range(Hq):
        np.testing.assert_allclose(out[0, h], h // 4 + 1, rtol=1e-14)
    # identical queries inside one group see identical keys -> identical rows
    q[0, 1] = q[0, 0]
    V = rng.standard_normal((L, Hkv, d)).astype(np.float32)
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    assert np.array_equal(out[0, 0], out[0, 1]) and lse[0, 0] == lse[0, 1]
    assert not np.array_equal(out[0, 0], out[0, 4])


def test_page_permutation_leaves_output_bit_identical():
    q, K, V = rand_case(7, 150, 8, 2, 64)
    res = []
    for perm_seed in (0, 1, 2):
        kp, vp, table, lens = tiny_cache(K, V, perm_seed=perm_seed, pool_extra=5)
        res.append(oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125))
    for o, l in res[1:]:
        assert np.array_equal(o, res[0][0]) and np.array_equal(l, res[0][1])


@pytest.mark.parametrize("L", [1, 15, 16, 17, 31, 32, 33])
def test_masked_slots_never_read(L):
    """Tails of last pages, unused pages and unassigned table entries hold NaN / -1."""
    q, K, V = rand_case(L, L, 4, 1, 64)
    kp, vp, table, lens = tiny_cache(K, V)  # pools start as all-NaN
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    assert np.all(np.isfinite(out)) and np.all(np.isfinite(lse))
    kz, vz = kp.copy(), vp.copy()
    kz[kz == wl.NAN_BF16_BITS] = 0
    vz[vz == wl.NAN_BF16_BITS] = 0
    o2, l2 = oracle.decode_attn(bf16(q), kz, vz, table, lens, 0.125)
    assert np.array_equal(out, o2) and np.array_equal(lse, l2)


def test_overflow_safety():
    d, L = 64, 20
    q = np.zeros((1, 1, d), np.float32); q[0, 0, 0] = 256.0
    K = np.zeros((L, 1, d), np.float32); K[7, 0, 0] = 32.0  # scaled logit 1024
    rng = np.random.default_rng(9)
    V = rng.standard_normal((L, 1, d)).astype(np.float32)
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    np.testing.assert_allclose(out[0, 0], oracle.bf16_bits_to_f64(bf16(V))[7, 0], rtol=1e-14, atol=1e-300)
    assert lse[0, 0] == pytest.approx(1024.0, rel=1e-14)
    K[:, 0, 0] = -32.0  # every logit -1024 -> uniform weights
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    np.testing.assert_allclose(out[0, 0], oracle.bf16_bits_to_f64(bf16(V))[:, 0].mean(axis=0), rtol=1e-13, atol=1e-16)
    assert lse[0, 0] == pytest.approx(-1024.0 + math.log(L), rel=1e-14)


def test_shift_invariance_with_exact_integer_inputs():
    """Adding c to every key moves every logit by scale*<q,c>: out unchanged, lse shifted."""
    rng = np.random.default_rng(11)
    d, L = 64, 33
    q = rng.integers(-3, 3, size=(1, 2, d), endpoint=True).astype(np.float32)
    K = rng.integers(-8, 8, size=(L, 1, d), endpoint=True).astype(np.float32)
    V = rng.standard_normal((L, 1, d)).astype(np.float32)
    c = rng.integers(-4, 4, size=(1, 1, d), endpoint=True).astype(np.float32)
    kp, vp, table, lens = tiny_cache(K, V)
    o1, l1 = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    kp2, vp2, table2, _ = tiny_cache(K + c, V)
    o2, l2 = oracle.decode_attn(bf16(q), kp2, vp2, table2, lens, 0.125)
    np.testing.assert_allclose(o1, o2, rtol=1e-12, atol=1e-15)
    for h in range(2):
        assert l2[0, h] - l1[0, h] == pytest.approx(0.125 * float(np.dot(q[0, h], c[0, 0])), abs=1e-11)


def test_output_is_a_convex_combination():
    q, K, V = rand_case(12, 77, 8, 2, 64)
    kp, vp, table, lens = tiny_cache(K, V)
    out, _ = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125)
    vb = oracle.bf16_bits_to_f64(bf16(V))
    for h in range(8):
        assert np.all(out[0, h] <= vb[:, h // 4].max(axis=0) + 1e-15)
        assert np.all(out[0, h] >= vb[:, h // 4].min(axis=0) - 1e-15)


def test_empty_context_and_token_ranges():
    q, K, V = rand_case(13, 40, 2, 1, 64)
    kp, vp, table, lens = tiny_cache(K, V)
    out, lse = oracle.decode_attn(bf16(q), kp, vp, table, np.array([0], np.int32), 0.125)
    assert np.all(out == 0.0) and np.all(lse == -np.inf)
    # a range equals attention over a cache that holds only those tokens
    o_r, l_r = oracle.decode_attn(bf16(q), kp, vp, table, lens, 0.125, t_begin=[5], t_end=[21])
    kp2, vp2, table2, lens2 = tiny_cache(K[5:21], V[5:21])
    o_s, l_s = oracle.decode_attn(bf16(q), kp2, vp2, table2, lens2, 0.125)
    np.testing.assert_allclose(o_r, o_s, rtol=1e-14)
    np.testing.assert_allclose(l_r, l_s, rtol=1e-14)


# ---------------------------------------------------------------- split + merge

def partials(qb, kp, vp, table, lens, cuts, scale):
    o_parts, l_parts = [], []
    for a, b in zip(cuts[:-1], cuts[1:]):
        o, l = oracle.decode_attn(qb, kp, vp, table, lens, scale, t_begin=[a], t_end=[b], nthreads=1)
        o_parts.append(o[0])
        l_parts.append(l[0])
    return np.stack(o_parts), np.stack(l_parts)  # [n, Hq, d], [n, Hq]


def test_every_partition_of_a_short_context_merges_to_the_unsplit_result():
    L = 10
    q, K, V = rand_case(14, L, 2, 1, 64)
    kp, vp, table, lens = tiny_cache(K, V)
    qb = bf16(q)
    full, full_lse = oracle.decode_attn(qb, kp, vp, table, lens, 0.125)
    count = 0
    for mask in range(1 << (L - 1)):  # each bit = a cut after token i
        cuts = [0] + [i + 1 for i in range(L - 1) if mask >> i & 1] + [L]
        op, lp = partials(qb, kp, vp, table, lens, cuts, 0.125)
        for h in range(2):
            om, lm = oracle.lse_merge(op[:, h], lp[:, h])
            np.testing.assert_allclose(om, full[0, h], rtol=1e-12, atol=1e-15)
            assert lm == pytest.approx(full_lse[0, h], rel=1e-13, abs=1e-13)
        count += 1
    assert count == 512


def test_random_partitions_of_long_contexts_and_empty_parts():
    rng = np.random.default_rng(15)
    for L in (257, 4096):
        q, K, V = rand_case(L, L, 4, 2, 64)
        kp, vp, table, lens = tiny_cache(K, V)
        qb = bf16(q)
        full, full_lse = oracle.decode_attn(qb, kp, vp, table, lens, 0.125)
        for _ in range(3):
            inner = np.sort(rng.choice(np.arange(1, L), size=7, replace=False)).tolist()
            cuts = [0] + inner + [L]
            cuts.insert(3, cuts[3])  # one empty part: lse = -inf, no weight
            op, lp = partials(qb, kp, vp, table, lens, cuts, 0.125)
            assert np.any(np.isinf(lp))
            for h in range(4):
                om, lm = oracle.lse_merge(op[:, h], lp[:, h])
                np.testing.assert_allclose(om, full[0, h], rtol=1e-12, atol=1e-15)
                assert lm == pytest.approx(full_lse[0, h], rel=1e-13)
    om, lm = oracle.lse_merge(np.zeros((2, 4)), np.array([-np.inf, -np.inf]))
    assert np.all(om == 0) and lm == -np.inf


def test_merge_weights_follow_exp_of_lse():
    # two parts with lse 0 and ln 3 -> weights 1/4 and 3/4
    o = np.array([[4.0, 0.0], [0.0, 4.0]])
    om, lm = oracle.lse_merge(o, np.array([0.0, math.log(3.0)]))
    np.testing.assert_allclose(om, [1.0, 3.0], rtol=1e-15)
    assert lm == pytest.approx(math.log(4.0), rel=1e-15)


# ---------------------------------------------------------------- append

def test_append_writes_exactly_the_addressed_bytes():
    Hkv, d, P = 2, 64, 16
    lens0 = np.array([0, 15, 16, 31, 47], dtype=np.int32)  # slot 0 of a fresh page, slot 15, ...
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=21, reserve_tokens=3)
    kp, vp = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    k_ref, v_ref = kp.copy(), vp.copy()
    lens = lens0.copy()
    table = cache.page_table_host
    for step in range(3):
        kn = oracle.bf16_bits(wl.random_bf16((5, Hkv, d), 100 + step))
        vn = oracle.bf16_bits(wl.random_bf16((5, Hkv, d), 200 + step))
        rc = oracle.kv_append(kn, vn, kp, vp, table, lens)
        assert rc == 0
        for b in range(5):  # independent index arithmetic on the mirror
            pos = lens0[b] + step
            k_ref[table[b, pos // P], :, pos % P, :] = kn[b]
            v_ref[table[b, pos // P], :, pos % P, :] = vn[b]
        assert np.array_equal(kp, k_ref) and np.array_equal(vp, v_ref)
        assert np.array_equal(lens, lens0 + step + 1)
    # without advance the lengths stay
    keep = lens.copy()
    oracle.kv_append(kn, vn, kp, vp, table, lens, advance=False)
    assert np.array_equal(lens, keep)


def test_append_rejects_out_of_range_without_writing():
    cache = wl.build_paged_cache(np.array([16], np.int32), 1, 64, seed=22)
    kp, vp = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    before = kp.copy()
    lens = np.array([16], np.int32)  # next page is unassigned (-1) or past the table
    kn = oracle.bf16_bits(wl.random_bf16((1, 1, 64), 1))
    table = np.full((1, 2), -1, np.int32)
    table[0, 0] = cache.page_table_host[0, 0]
    assert oracle.kv_append(kn, kn, kp, vp, table, lens) == -1
    assert np.array_equal(kp, before) and lens[0] == 16


def test_appended_token_is_visible_to_the_next_attention():
    """Append first, then attend over old_len + 1 tokens: a key aligned with q takes all the weight."""
    Hq, Hkv, d = 4, 1, 64
    lens = np.array([30], np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=23, reserve_tokens=1)
    kp, vp = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    q = wl.random_bf16((1, Hq, d), 5)
    q[0, 1:] = q[0, 0]
    k_new = (64.0 * q[:, :1].float()).to(torch.bfloat16)  # one KV head, aligned with every query head
    v_new = wl.random_bf16((1, Hkv, d), 6)
    cur = lens.copy()
    oracle.kv_append(oracle.bf16_bits(k_new), oracle.bf16_bits(v_new), kp, vp, cache.page_table_host, cur)
    assert cur[0] == 31
    out, _ = oracle.decode_attn(oracle.bf16_bits(q), kp, vp, cache.page_table_host, cur, 0.125)
    np.testing.assert_allclose(out[0, 0], v_new[0, 0].double().numpy(), atol=1e-9)


def test_workload_length_recipes():
    for cfg, lo, hi in ((0, 16, 256), (1, 2048, 16384), (2, 1024, 32768), (3, 32768, 65536), (4, 256, 40960)):
        lens = wl.context_lengths(cfg)
        assert len(lens) == wl.WORKLOADS[cfg].batch and lens.min() >= lo and lens.max() <= hi
        assert np.array_equal(lens, wl.context_lengths(cfg))  # seeded
    assert abs(np.median(wl.context_lengths(2, batch=20000)) - 8192) < 300
    parts = wl.shard_sequences(wl.context_lengths(1), 2)
    assert sorted(np.concatenate(parts).tolist()) == list(range(64))
    tok = [int(wl.context_lengths(1)[p].sum()) for p in parts]
    assert abs(tok[0] - tok[1]) < 16384
    assert len(list(itertools.chain(*parts))) == 64


# ---------------------------------------------------------------- KV page gather / scatter

def test_gather_matches_fancy_indexing_and_scatter_inverts_it():
    Hkv, d, P = 2, 64, 16
    lens = np.array([100, 16, 33, 0, 250], dtype=np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=30)
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    table = cache.page_table_host
    pages = (lens + P - 1) // P
    pb = np.array([2, 0, 1, 0, 5], dtype=np.int32)             # only the pages of the "new" tokens
    pe = pages.astype(np.int32)
    cnt = np.maximum(pe - pb, 0)
    off = np.concatenate([[0], np.cumsum(cnt)[:-1]]).astype(np.int64)
    packed, rc = oracle.kv_gather(kp, vp, table, pb, pe, off, int(cnt.sum()))
    assert rc == 0
    for b in range(5):  # independent statement with NumPy fancy indexing
        ids = table[b, pb[b]:pe[b]]
        assert np.array_equal(packed[off[b]:off[b] + cnt[b], 0], kp[ids])
        assert np.array_equal(packed[off[b]:off[b] + cnt[b], 1], vp[ids])
    # scatter into a differently permuted destination cache, then compare logical contents
    dst = wl.build_paged_cache(lens, Hkv, d, seed=31)
    dk, dv = oracle.bf16_bits(dst.k_pages).copy(), oracle.bf16_bits(dst.v_pages).copy()
    before_k = dk.copy()
    assert oracle.kv_scatter(packed, off, dk, dv, dst.page_table_host, pb, pe) == 0
    touched = np.zeros(dk.shape[0], dtype=bool)
    for b in range(5):
        src_ids, dst_ids = table[b, pb[b]:pe[b]], dst.page_table_host[b, pb[b]:pe[b]]
        assert np.array_equal(dk[dst_ids], kp[src_ids]) and np.array_equal(dv[dst_ids], vp[src_ids])
        touched[dst_ids] = True
    assert np.array_equal(dk[~touched], before_k[~touched])  # nothing else was written
    # an unassigned page id is reported and skipped
    bad = table.copy()
    bad[0, 3] = -1
    _, rc = oracle.kv_gather(kp, vp, bad, pb, pe, off, int(cnt.sum()))
    assert rc == -1


# ---------------------------------------------------------------- append-prefill attention

def prefill_case(seed, lens, q_lens, Hq, Hkv, d):
    lens, q_lens = np.asarray(lens, np.int32), np.asarray(q_lens, np.int32)
    cache = wl.build_paged_cache(lens, Hkv, d, seed=seed, poison=True)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    q = oracle.bf16_bits(wl.random_bf16((int(ip[-1]), Hq, d), seed + 1))
    return cache, ip, q


def test_prefill_equals_decode_definition_per_token_and_sdpa_causal():
    Hq, Hkv, d = 4, 2, 64
    lens, q_lens = [70, 33, 5, 40], [20, 33, 1, 0]
    cache, ip, q = prefill_case(60, lens, q_lens, Hq, Hkv, d)
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    out, lse = oracle.prefill_attn(q, ip, kp, vp, cache.page_table_host, np.asarray(lens, np.int32), 0.125)
    assert np.all(np.isfinite(out)) and out.shape[0] == 54
    kf, vf = oracle.bf16_bits_to_f64(kp), oracle.bf16_bits_to_f64(vp)
    for b in range(4):
        L, n = lens[b], q_lens[b]
        if n == 0:
            continue
        # (1) every query token as a decode query over its visible prefix (the pinned decode definition)
        for i in range(n):
            vis = np.array([L - n + i + 1], np.int32)
            o1, l1 = oracle.decode_attn(q[ip[b] + i][None], kp, vp, cache.page_table_host[b][None], vis, 0.125)
            np.testing.assert_allclose(out[ip[b] + i], o1[0], rtol=1e-13, atol=1e-15)
            np.testing.assert_allclose(lse[ip[b] + i], l1[0], rtol=1e-13)
        # (2) torch SDPA on the dense layout with an explicit bottom-right-aligned causal mask
        t = np.arange(L)
        pages = cache.page_table_host[b, t // 16]
        for kvh in range(Hkv):
            Kd = torch.from_numpy(kf[pages, kvh, t % 16])      # [L, d]
            Vd = torch.from_numpy(vf[pages, kvh, t % 16])
            for h in range(kvh * 2, kvh * 2 + 2):
                Qd = torch.from_numpy(oracle.bf16_bits_to_f64(q[ip[b]:ip[b + 1], h]))  # [n, d]
                mask = torch.arange(L)[None, :] <= (L - n + torch.arange(n))[:, None]
                ref = torch.nn.functional.scaled_dot_product_attention(Qd[None], Kd[None], Vd[None], attn_mask=mask[None],
                                                                       scale=0.125)[0].numpy()
                np.testing.assert_allclose(out[ip[b]:ip[b + 1], h], ref, rtol=1e-12, atol=1e-14)


def test_prefill_first_token_of_a_fresh_sequence_sees_only_itself():
    Hq, Hkv, d = 2, 1, 64
    cache, ip, q = prefill_case(61, [19], [19], Hq, Hkv, d)
    kp, vp = oracle.bf16_bits(cache.k_pages), oracle.bf16_bits(cache.v_pages)
    out, lse = oracle.prefill_attn(q, ip, kp, vp, cache.page_table_host, np.array([19], np.int32), 0.125)
    v0 = oracle.bf16_bits_to_f64(vp)[cache.page_table_host[0, 0], 0, 0]
    for h in range(Hq):
        assert np.array_equal(out[0, h], v0)
    # the last query sees everything: equal to plain decode attention over the whole context
    o1, _ = oracle.decode_attn(q[18][None], kp, vp, cache.page_table_host, np.array([19], np.int32), 0.125)
    np.testing.assert_allclose(out[18], o1[0], rtol=1e-13)
    # future tokens never leak: changing the last token's K/V leaves every earlier row untouched
    kp2, vp2 = kp.copy(), vp.copy()
    page = cache.page_table_host[0, 1]
    kp2[page, :, 2] = bf16(np.full((Hkv, d), 3.0)); vp2[page, :, 2] = bf16(np.full((Hkv, d), -5.0))  # token 18
    out2, _ = oracle.prefill_attn(q, ip, kp2, vp2, cache.page_table_host, np.array([19], np.int32), 0.125)
    assert np.array_equal(out2[:18], out[:18]) and not np.array_equal(out2[18], out[18])


def test_multi_token_append_then_prefill_matches_token_by_token_decode():
    """Appending a turn at once and prefilling equals appending one token at a time and decoding."""
    Hq, Hkv, d = 4, 1, 64
    lens0 = np.array([30, 0, 16], np.int32)
    q_lens = np.array([5, 18, 16], np.int32)
    cache = wl.build_paged_cache(lens0, Hkv, d, seed=62, reserve_tokens=20)
    ip = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    total = int(ip[-1])
    kn = oracle.bf16_bits(wl.random_bf16((total, Hkv, d), 63))
    vn = oracle.bf16_bits(wl.random_bf16((total, Hkv, d), 64))
    q = oracle.bf16_bits(wl.random_bf16((total, Hq, d), 65))
    kp, vp = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    lens = lens0.copy()
    assert oracle.kv_append_tokens(kn, vn, ip, kp, vp, cache.page_table_host, lens) == 0
    assert np.array_equal(lens, lens0 + q_lens)
    out, _ = oracle.prefill_attn(q, ip, kp, vp, cache.page_table_host, lens, 0.125)
    # token by token with the single-token append and the decode definition
    kp1, vp1 = oracle.bf16_bits(cache.k_pages).copy(), oracle.bf16_bits(cache.v_pages).copy()
    for b in range(3):
        cur = np.array([lens0[b]], np.int32)
        for i in range(q_lens[b]):
            r = ip[b] + i
            oracle.kv_append(kn[r][None], vn[r][None], kp1, vp1, cache.page_table_host[b][None], cur)
            o1, _ = oracle.decode_attn(q[r][None], kp1, vp1, cache.page_table_host[b][None], cur, 0.125)
            np.testing.assert_allclose(out[r], o1[0], rtol=1e-13, atol=1e-15)
    assert np.array_equal(kp, kp1) and np.array_equal(vp, vp1)

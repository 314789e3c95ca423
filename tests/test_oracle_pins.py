"""Pins of the CPU oracle against what the paper and the mathematics fix.

None of these tests touches the CUDA library.  Each pin is chosen so that a
plausible mistake in the oracle (dropped term, wrong sign or index, transposed
operand, wrong tie-break, wrong eviction order) fails at least one of them.
"""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest

import dip_inputs as di
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _mat_f32(a):
    a = np.ascontiguousarray(a, dtype=np.float32)
    return oracle.Matrix(oracle.W_F32, a, None, a.shape[0], a.shape[1])


def _rand_layer(seed, d_model, d_ff, wtype=di.W_F32):
    w = di.WORKLOADS["block_f32"].scaled(seed=seed, d_model=d_model, d_ff=d_ff, wtype=wtype)
    return di.layer_weights(w, 0)


def _oracle_mats(lw):
    t = lw.wtype
    return (oracle.Matrix(t, lw.gate, lw.gate_scales, lw.d_ff, lw.d_model),
            oracle.Matrix(t, lw.up, lw.up_scales, lw.d_ff, lw.d_model),
            oracle.Matrix(t, lw.down, lw.down_scales, lw.d_model, lw.d_ff))


def _to_f64(lw):
    """Decode stored weights to float64 with numpy only (format definitions)."""
    if lw.wtype == di.W_F32:
        return [a.astype(np.float64) for a in (lw.gate, lw.up, lw.down)]
    if lw.wtype == di.W_BF16:
        return [di.bf16_bits_to_f32(a).astype(np.float64) for a in (lw.gate, lw.up, lw.down)]
    return [di.dequantize_int4_g128(a, s, *shape).astype(np.float64)
            for a, s, shape in ((lw.gate, lw.gate_scales, (lw.d_ff, lw.d_model)),
                                (lw.up, lw.up_scales, (lw.d_ff, lw.d_model)),
                                (lw.down, lw.down_scales, (lw.d_model, lw.d_ff)))]


# --------------------------------------------------------------------------
# SiLU (Eq. 2)
# --------------------------------------------------------------------------
def test_silu_closed_forms():
    assert oracle.silu(0.0) == 0.0
    for z in [0.1, 0.5, 1.0, 2.0, 3.75, 10.0, 30.0]:
        # silu(z) - silu(-z) = z  (sigmoid(z) + sigmoid(-z) = 1)
        assert oracle.silu(z) - oracle.silu(-z) == pytest.approx(z, rel=1e-15)
        # z * sigmoid(z) with sigmoid written through tanh
        assert oracle.silu(z) == pytest.approx(z * 0.5 * (1.0 + math.tanh(0.5 * z)), rel=1e-14)
    assert oracle.silu(1.0) == pytest.approx(0.7310585786300049, rel=1e-15)
    assert oracle.silu(-40.0) == pytest.approx(-40.0 * math.exp(-40.0), rel=1e-12)
    assert oracle.silu(40.0) == pytest.approx(40.0, rel=1e-15)
    # global minimum of silu is about -0.27846 at z about -1.27846
    zs = np.linspace(-3, 0, 3001)
    vals = [oracle.silu(float(z)) for z in zs]
    assert min(vals) == pytest.approx(-0.2784645427610738, abs=1e-7)


def test_glu_elementwise_pins():
    """Eq. 2 for given pre-activations: u * silu(g).  Closed forms, the tanh form of the sigmoid,
    oddness in u, and the dense oracle's GLU on the same pre-activations."""
    g = np.array([0.0, 1.0, -1.0, 40.0, -40.0, 2.5], dtype=np.float64)
    u = np.array([3.0, 2.0, 2.0, -1.5, 7.0, 0.0], dtype=np.float64)
    h = oracle.glu(g, u)
    assert h[0] == 0.0 and h[5] == 0.0
    assert h[1] == pytest.approx(2.0 * 0.7310585786300049, rel=1e-15)
    assert h[1] - h[2] == pytest.approx(2.0 * 1.0, rel=1e-15)       # silu(z) - silu(-z) = z, times u
    assert h[3] == pytest.approx(-1.5 * 40.0, rel=1e-15)
    assert h[4] == pytest.approx(7.0 * -40.0 * math.exp(-40.0), rel=1e-12)
    rng = np.random.default_rng(8)
    g, u = rng.standard_normal(200) * 3, rng.standard_normal(200)
    np.testing.assert_allclose(oracle.glu(g, u), u * g * 0.5 * (1.0 + np.tanh(0.5 * g)), rtol=1e-11, atol=1e-15)
    np.testing.assert_array_equal(oracle.glu(g, -u), -oracle.glu(g, u))
    assert not np.allclose(oracle.glu(g, u), oracle.glu(u, g))           # the gate is the activated branch
    lw = _rand_layer(21, 64, 96)
    Wg, Wu, Wd = _oracle_mats(lw)
    x = di.heavy_tail_vector(22, 64)
    ones = np.ones(64, dtype=np.uint8)
    glu_dense, _ = oracle.dense_mlp(Wg, Wu, Wd, x)
    np.testing.assert_array_equal(oracle.glu(oracle.masked_matvec(Wg, x, ones), oracle.masked_matvec(Wu, x, ones)),
                                  glu_dense)


# --------------------------------------------------------------------------
# stored formats
# --------------------------------------------------------------------------
def test_weight_decoding_bf16_and_int4_against_numpy():
    rng = np.random.default_rng(5)
    w = (rng.standard_normal((6, 256)) * 0.02).astype(np.float32)
    bits = di.f32_to_bf16_bits(w)
    M = oracle.Matrix(oracle.W_BF16, bits, None, 6, 256)
    ref = di.bf16_bits_to_f32(bits)
    for j, i in [(0, 0), (5, 255), (2, 17), (3, 128)]:
        assert M.element(j, i) == float(ref[j, i])
    # bf16 rounding is to nearest: relative error at most 2^-8 (8-bit significand)
    assert np.max(np.abs(ref - w) / np.abs(w)) <= 2.0 ** -8
    q, s = di.quantize_int4_g128(w)
    Mq = oracle.Matrix(oracle.W_INT4_G128, q, s, 6, 256)
    deq = di.dequantize_int4_g128(q, s, 6, 256)
    for j in range(6):
        for i in [0, 1, 2, 127, 128, 129, 254, 255]:
            assert Mq.element(j, i) == float(deq[j, i])
    # symmetric 4-bit with scale max/7: error at most half a step
    step = s.view(np.float16).astype(np.float64).T  # [d_out, groups]
    err = np.abs(deq.astype(np.float64) - w).reshape(6, 2, 128).max(axis=2)
    assert np.all(err <= 0.5 * step * (1 + 1e-3) + 1e-12)


def test_fp16_scale_decoding_special_values():
    # scale bit patterns: 1.0, 2^-14 (smallest normal), 2^-24 (smallest subnormal), 0.333251953125
    pats = np.array([0x3C00, 0x0400, 0x0001, 0x3555], dtype=np.uint16)
    expect = pats.view(np.float16).astype(np.float64)
    q = np.full((4, 64), 0x99, dtype=np.uint8)  # both nibbles 9 -> +1
    s = pats.reshape(1, 4).copy()
    M = oracle.Matrix(oracle.W_INT4_G128, q, s, 4, 128)
    for j in range(4):
        assert M.element(j, 3) == expect[j]


# --------------------------------------------------------------------------
# dense MLP (Eq. 1-2) against a library matmul
# --------------------------------------------------------------------------
@pytest.mark.parametrize("wtype", [di.W_F32, di.W_BF16, di.W_INT4_G128])
def test_dense_mlp_against_numpy(wtype):
    lw = _rand_layer(11, 128, 384, wtype)
    Wg, Wu, Wd = _to_f64(lw)
    x = di.heavy_tail_vector(3, 128)
    g = Wg @ x.astype(np.float64)
    u = Wu @ x.astype(np.float64)
    glu_ref = u * (g / (1.0 + np.exp(-g)))
    y_ref = Wd @ glu_ref
    glu, y = oracle.dense_mlp(*_oracle_mats(lw), x)
    np.testing.assert_allclose(glu, glu_ref, rtol=1e-11, atol=1e-15)
    np.testing.assert_allclose(y, y_ref, rtol=1e-10, atol=1e-14)
    # the gate goes through the non-linearity, not the up branch: swapping them must differ
    glu_swapped = g * (u / (1.0 + np.exp(-u)))
    assert np.max(np.abs(glu - glu_swapped)) > 1e-3


def test_keep_ratio_one_reproduces_dense_exactly():
    lw = _rand_layer(12, 96, 160)
    mats = _oracle_mats(lw)
    x = di.heavy_tail_vector(4, 96)
    glu, y = oracle.dense_mlp(*mats, x)
    r = oracle.mlp_step(*mats, x, 96, 160)
    assert r.m_x.sum() == 96 and r.m_h.sum() == 160
    # h is carried in binary32 between the halves
    np.testing.assert_array_equal(r.h32, glu.astype(np.float32))
    y_from_h32 = lw.down.astype(np.float64) @ r.h32.astype(np.float64)
    np.testing.assert_allclose(r.y, y_from_h32, rtol=1e-12, atol=1e-16)
    np.testing.assert_allclose(r.y, y, rtol=1e-5, atol=1e-9)


def test_glu_pruning_is_dip_with_dense_gate_up():
    """Eq. 4: pruning only GLU(x) (dense gate/up) equals the step with k_x = d_model."""
    lw = _rand_layer(13, 64, 192)
    Wg, Wu, Wd = _to_f64(lw)
    x = di.heavy_tail_vector(5, 64)
    g = Wg @ x.astype(np.float64)
    u = Wu @ x.astype(np.float64)
    glu = (u * (g / (1.0 + np.exp(-g)))).astype(np.float32)
    k_h = 48
    order = sorted(range(192), key=lambda i: (-abs(float(glu[i])), i))[:k_h]
    m = np.zeros(192)
    m[order] = 1
    y_ref = Wd @ (glu.astype(np.float64) * m)
    r = oracle.mlp_step(*_oracle_mats(lw), x, 64, k_h)
    assert set(np.nonzero(r.m_h)[0]) == set(order)
    np.testing.assert_allclose(r.y, y_ref, rtol=1e-9, atol=1e-13)


# --------------------------------------------------------------------------
# hand-worked example
# --------------------------------------------------------------------------
def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            k, v = line.split(":", 1)
            out[k.strip()] = [float(t) for t in v.split()]
    return out


def test_hand_worked_step():
    g = _read_golden("tiny_step.txt")
    x = np.array(g["x"], dtype=np.float32)
    Wg = _mat_f32(np.array(g["Wg"]).reshape(3, 4))
    Wu = _mat_f32(np.array(g["Wu"]).reshape(3, 4))
    Wd = _mat_f32(np.array(g["Wd"]).reshape(4, 3))
    r = oracle.mlp_step(Wg, Wu, Wd, x, int(g["k_x"][0]), int(g["k_h"][0]))
    assert r.m_x.tolist() == [int(v) for v in g["m_x"]]
    assert r.idx_x.tolist() == [1, 3]
    np.testing.assert_allclose(r.h32, np.array(g["h"]), rtol=1e-7)
    assert r.m_h.tolist() == [int(v) for v in g["m_h"]]
    assert r.idx_h.tolist() == [1, 2]
    np.testing.assert_allclose(r.y, np.array(g["y"]), rtol=2e-7)


def test_hand_worked_cache_aware_call():
    g = _read_golden("tiny_step.txt")
    x = np.array(g["x"], dtype=np.float32)
    c = np.array(g["ca_c"], dtype=np.uint8)
    gamma = g["ca_gamma"][0]
    np.testing.assert_allclose(oracle.ca_score(x, c, gamma), np.array(g["ca_s"]), rtol=1e-15)
    cache = oracle.Cache(4, 2)
    cache.stamp[:] = np.where(c > 0, 0, -1)
    cache.n_resident[0] = 2
    m, idx = oracle.dip_ca_mask(x, 2, gamma, cache)
    assert m.tolist() == [int(v) for v in g["ca_m"]]
    assert cache.resident().tolist() == [int(v) for v in g["ca_resident_after"]]
    assert cache.counters.tolist() == [int(v) for v in g["ca_counters"]]
    assert cache.n_resident[0] == 2 and cache.step[0] == 1


# --------------------------------------------------------------------------
# top-k (Sec. 3.1)
# --------------------------------------------------------------------------
def _topk_bruteforce(keys, k):
    """O(d^2) rank count: column i is kept iff fewer than k columns precede it in
    (key descending, index ascending) order."""
    d = len(keys)
    m = []
    for i in range(d):
        before = sum(1 for j in range(d) if keys[j] > keys[i] or (keys[j] == keys[i] and j < i))
        m.append(1 if before < k else 0)
    return m


def test_topk_exhaustive_small_alphabet():
    for d in range(1, 8):
        for vec in itertools.product((0, 1, 5), repeat=d):
            keys = np.array(vec, dtype=np.uint32)
            for k in range(0, d + 1):
                m, idx = oracle.topk_mask(keys, k)
                assert m.tolist() == _topk_bruteforce(vec, k)
                assert idx.tolist() == [i for i in range(d) if m[i]]


def test_topk_all_permutations():
    for d in range(1, 8):
        for perm in itertools.permutations(range(d)):
            keys = np.array(perm, dtype=np.uint32) * 7 + 3
            for k in (0, 1, d // 2, d - 1, d):
                if k < 0:
                    continue
                m, _ = oracle.topk_mask(keys, k)
                assert sorted(np.nonzero(m)[0].tolist()) == sorted(i for i in range(d) if perm[i] >= d - k)


def test_topk_random_with_duplicates_and_properties():
    rng = np.random.default_rng(0)
    for trial in range(300):
        d = int(rng.integers(1, 17))
        keys = rng.integers(0, 6, size=d).astype(np.uint32)
        k = int(rng.integers(0, d + 1))
        m, idx = oracle.topk_mask(keys, k)
        assert m.tolist() == _topk_bruteforce(keys.tolist(), k)
    x = di.heavy_tail_vector(9, 4096)
    x[100:140] = x[7]           # a block of exact ties
    x[200] = -x[7]              # sign does not matter
    x[300] = 0.0
    x[301] = -0.0
    for k in (1, 37, 1024, 4095, 4096):
        m, idx = oracle.dip_ca_mask(x, k)
        assert int(m.sum()) == k and len(idx) == k
        assert np.all(np.diff(idx) > 0)
        a = np.abs(x)
        if k < 4096:
            assert a[m == 1].min() >= a[m == 0].max()
            thr = a[m == 1].min()
            tied_kept = np.nonzero((a == thr) & (m == 1))[0]
            tied_dropped = np.nonzero((a == thr) & (m == 0))[0]
            if len(tied_dropped):
                assert tied_kept.max() < tied_dropped.min()      # lower index wins a tie
    assert oracle.dip_ca_mask(np.zeros(8, np.float32), 3)[1].tolist() == [0, 1, 2]
    with pytest.raises(ValueError):
        oracle.topk_mask(np.zeros(4, np.uint32), 5)


def test_rank_key_is_binary32_product_bits():
    assert oracle.rank_key(-0.0, True, 0.2) == 0
    assert oracle.rank_key(1.5, True, 0.2) == int(np.float32(1.5).view(np.uint32))
    rng = np.random.default_rng(1)
    for v in rng.standard_normal(200).astype(np.float32):
        p = np.float32(abs(v)) * np.float32(0.2)
        assert oracle.rank_key(float(v), False, 0.2) == int(np.float32(p).view(np.uint32))
        # exact product rounded once to binary32 (Fraction arithmetic, then nearest float)
        exact = Fraction(float(np.float32(abs(v)))) * Fraction(float(np.float32(0.2)))
        assert float(p) == float(np.float32(float(exact)))
    # keys order like the magnitudes
    a, b = np.float32(1e-30), np.float32(3.0)
    assert oracle.rank_key(float(a), True, 1.0) < oracle.rank_key(float(b), True, 1.0)


# --------------------------------------------------------------------------
# cache-aware score (Eq. 10) and Alg. 1
# --------------------------------------------------------------------------
def _exact_ca_mask(x, c, gamma, k):
    """Eq. 10 in exact rational arithmetic, normalisation included, then top-k
    with the lower index winning ties."""
    xs = [abs(Fraction(float(v))) for v in x]
    norm = max(xs)
    g = Fraction(gamma)
    s = [(xi * (1 if ci else g)) / norm if norm else Fraction(0) for xi, ci in zip(xs, c)]
    order = sorted(range(len(x)), key=lambda i: (-s[i], i))[:k]
    m = [0] * len(x)
    for i in order:
        m[i] = 1
    return m, s


def test_ca_mask_equals_exact_rational_ranking():
    rng = np.random.default_rng(2)
    for trial in range(400):
        d = int(rng.integers(2, 13))
        # dyadic magnitudes and dyadic gamma: every product is exact in binary32
        x = (rng.integers(-32, 33, size=d) / 8.0).astype(np.float32)
        gamma = float(rng.choice([0.0, 0.125, 0.25, 0.5, 1.0]))
        c = rng.integers(0, 2, size=d).astype(np.uint8)
        k = int(rng.integers(1, d + 1))
        cache = oracle.Cache(d, d)
        cache.stamp[:] = np.where(c > 0, 0, -1)
        cache.n_resident[0] = int(c.sum())
        m, _ = oracle.dip_ca_mask(x, k, gamma, cache)
        m_ref, s_ref = _exact_ca_mask(x, c, gamma, k)
        assert m.tolist() == m_ref
        s = oracle.ca_score(x, c, gamma)
        np.testing.assert_allclose(s, [float(v) for v in s_ref], rtol=1e-15)
        assert s.max() <= 1.0


def test_ca_reduces_to_dip():
    rng = np.random.default_rng(3)
    x = di.heavy_tail_vector(21, 512)
    m_dip, _ = oracle.dip_ca_mask(x, 128)
    for pattern in ("random", "ones", "zeros"):
        cache = oracle.Cache(512, 512)
        c = {"random": rng.integers(0, 2, 512), "ones": np.ones(512), "zeros": np.zeros(512)}[pattern]
        cache.stamp[:] = np.where(c > 0, 0, -1)
        cache.n_resident[0] = int((c > 0).sum())
        # gamma = 1: the penalty vanishes, any cache state
        m, _ = oracle.dip_ca_mask(x, 128, 1.0, cache.copy())
        np.testing.assert_array_equal(m, m_dip)
        if pattern == "ones":
            # all columns resident: uniform weight 1
            m, _ = oracle.dip_ca_mask(x, 128, 0.2, cache.copy())
            np.testing.assert_array_equal(m, m_dip)
        if pattern == "zeros":
            # nothing resident: uniform weight gamma; a power of two keeps the order exactly
            m, _ = oracle.dip_ca_mask(x, 128, 0.25, cache.copy())
            np.testing.assert_array_equal(m, m_dip)


def test_ca_scale_invariance_and_gamma_zero_and_monotonicity():
    rng = np.random.default_rng(4)
    x = di.heavy_tail_vector(22, 256)
    c = rng.integers(0, 2, 256).astype(np.uint8)

    def run(xv, gamma, cvec):
        cache = oracle.Cache(256, 256)
        cache.stamp[:] = np.where(cvec > 0, 0, -1)
        cache.n_resident[0] = int(cvec.sum())
        m, _ = oracle.dip_ca_mask(xv, 64, gamma, cache)
        return m, cache

    m0, _ = run(x, 0.2, c)
    for e in (-20, -3, 5, 30):
        m1, _ = run(np.ldexp(x, e).astype(np.float32), 0.2, c)
        np.testing.assert_array_equal(m0, m1)
    # gamma = 0 with at least k resident non-zero columns: every kept column is a hit
    assert int(((c > 0) & (x != 0)).sum()) >= 64
    mz, cz = run(x, 0.0, c)
    assert cz.counters[0] == 64 and cz.counters[1] == 0
    assert np.all(c[mz == 1] == 1)
    # cache-aware masking never has fewer hits than DIP on the same state
    m_dip, c_dip = run(x, 1.0, c)
    _, c_ca = run(x, 0.2, c)
    assert c_ca.counters[0] >= c_dip.counters[0]
    # making one more kept column resident never removes it from the mask
    kept_nonres = [i for i in range(256) if m0[i] and not c[i]]
    for i in kept_nonres[:10]:
        c2 = c.copy()
        c2[i] = 1
        m2, _ = run(x, 0.2, c2)
        assert m2[i] == 1


# --------------------------------------------------------------------------
# LRU column cache (Sec. 5.1) against an independent ordered-list replay
# --------------------------------------------------------------------------
class ListLRU:
    """Textbook LRU as an ordered list (front = least recently used).  A step's
    columns are processed one by one in ascending index; a column of the
    current step is never chosen as a victim; a miss that finds no victim is
    used without being cached."""

    def __init__(self, capacity):
        self.cap = capacity
        self.order = []
        self.hits = self.misses = self.evictions = self.bypassed = 0

    def step(self, cols):
        cols = sorted(cols)
        pinned = set(cols)
        before = set(self.order)
        for c in cols:
            if c in before:
                self.hits += 1
                self.order.remove(c)
                self.order.append(c)
                continue
            self.misses += 1
            if len(self.order) < self.cap:
                self.order.append(c)
                continue
            victim = next((v for v in self.order if v not in pinned), None)
            if victim is None:
                self.bypassed += 1
                continue
            self.order.remove(victim)
            self.evictions += 1
            self.order.append(c)


@pytest.mark.parametrize("d,cap", [(6, 0), (6, 2), (6, 6), (9, 4), (12, 5), (16, 8), (16, 3), (16, 16)])
def test_lru_matches_ordered_list_replay(d, cap):
    rng = np.random.default_rng(100 * d + cap)
    for trace in range(40):
        cache = oracle.Cache(d, cap)
        ref = ListLRU(cap)
        for t in range(30):
            k = int(rng.integers(0, d + 1)) if trace % 2 else int(rng.integers(1, max(2, d // 2)))
            cols = rng.choice(d, size=k, replace=False)
            m = np.zeros(d, dtype=np.uint8)
            m[cols] = 1
            was_resident = cache.resident()
            n_before = int(cache.n_resident[0])
            ctr_before = cache.counters.copy()
            oracle.cache_update(cache, m)
            ref.step(cols.tolist())
            assert sorted(np.nonzero(cache.resident())[0].tolist()) == sorted(ref.order)
            assert cache.counters.tolist() == [ref.hits, ref.misses, ref.evictions, ref.bypassed]
            # the list order (LRU first) is the (stamp, index) order of the stamps
            by_stamp = sorted(ref.order, key=lambda c: (cache.stamp[c], c))
            assert by_stamp == ref.order
            # invariants
            dh, dm, de, db = (cache.counters - ctr_before).tolist()
            assert dh + dm == k
            assert dh == int((m & was_resident).sum())
            assert int(cache.n_resident[0]) == int(cache.resident().sum()) <= cap
            assert dm == (int(cache.n_resident[0]) - n_before + de) + db
            if k <= cap:
                assert db == 0 and np.all(cache.resident()[m == 1] == 1)
            assert cache.step[0] == t + 1


def test_lru_fills_to_capacity_and_evicts_oldest():
    cache = oracle.Cache(8, 3)
    for cols in ([0], [1], [2]):
        m = np.zeros(8, np.uint8)
        m[cols] = 1
        oracle.cache_update(cache, m)
    assert cache.resident().tolist() == [1, 1, 1, 0, 0, 0, 0, 0]
    m = np.zeros(8, np.uint8)
    m[[0, 5]] = 1                     # 0 is refreshed, 5 replaces the oldest other column (1)
    oracle.cache_update(cache, m)
    assert cache.resident().tolist() == [1, 0, 1, 0, 0, 1, 0, 0]
    assert cache.counters.tolist() == [1, 4, 1, 0]
    with pytest.raises(ValueError):
        oracle.cache_update(oracle.Cache(4, 5), np.zeros(4, np.uint8))


# --------------------------------------------------------------------------
# masked mat-vec (Eq. 3, 7, 8)
# --------------------------------------------------------------------------
def test_masked_matvec_equals_dense_on_masked_input():
    rng = np.random.default_rng(6)
    W = (rng.standard_normal((40, 72)) * 0.02).astype(np.float32)   # non-square: a transpose cannot pass
    v = di.heavy_tail_vector(7, 72)
    m = (rng.random(72) < 0.3).astype(np.uint8)
    out = oracle.masked_matvec(_mat_f32(W), v, m)
    ref = W.astype(np.float64) @ (v.astype(np.float64) * m)
    np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-18)
    # one kept column i: the result is v_i times that column
    for i in (0, 13, 71):
        e = np.zeros(72, np.uint8)
        e[i] = 1
        np.testing.assert_array_equal(oracle.masked_matvec(_mat_f32(W), v, e),
                                      W[:, i].astype(np.float64) * float(v[i]))
    # linearity in v (exact for power-of-two scaling)
    np.testing.assert_array_equal(oracle.masked_matvec(_mat_f32(W), (4 * v).astype(np.float32), m), 4 * out)
    # empty mask
    assert not oracle.masked_matvec(_mat_f32(W), v, np.zeros(72, np.uint8)).any()


@pytest.mark.parametrize("wtype", [di.W_BF16, di.W_INT4_G128])
def test_sparse_step_on_stored_formats_equals_step_on_decoded_fp32(wtype):
    lw = _rand_layer(14, 256, 384, wtype)
    Wg, Wu, Wd = _to_f64(lw)
    x = di.heavy_tail_vector(8, 256)
    r = oracle.mlp_step(*_oracle_mats(lw), x, 64, 96)
    r32 = oracle.mlp_step(_mat_f32(Wg), _mat_f32(Wu), _mat_f32(Wd), x, 64, 96)
    np.testing.assert_array_equal(r.m_x, r32.m_x)
    np.testing.assert_array_equal(r.h32, r32.h32)
    np.testing.assert_array_equal(r.m_h, r32.m_h)
    np.testing.assert_array_equal(r.y, r32.y)
    # and against numpy on the masked inputs
    g = Wg @ (x.astype(np.float64) * r.m_x)
    u = Wu @ (x.astype(np.float64) * r.m_x)
    h = (u * g / (1 + np.exp(-g))).astype(np.float32)
    np.testing.assert_allclose(r.h32, h, rtol=1e-6, atol=1e-12)
    np.testing.assert_allclose(r.y, Wd @ (r.h32.astype(np.float64) * r.m_h), rtol=1e-10, atol=1e-15)


def test_step_with_caches_is_composition_of_alg1_calls():
    lw = _rand_layer(15, 128, 256)
    mats = _oracle_mats(lw)
    w = di.WORKLOADS["block_f32"].scaled(seed=15, d_model=128)
    xs = di.token_inputs(w, n_tokens=12, batch=1)[:, 0]
    cgu, cd = oracle.Cache(128, 64), oracle.Cache(256, 100)
    cgu2, cd2 = oracle.Cache(128, 64), oracle.Cache(256, 100)
    for x in xs:
        r = oracle.mlp_step(*mats, x, 32, 64, 0.2, cgu, cd)
        m_x, _ = oracle.dip_ca_mask(x, 32, 0.2, cgu2)
        np.testing.assert_array_equal(r.m_x, m_x)
        m_h, _ = oracle.dip_ca_mask(r.h32, 64, 0.2, cd2)
        np.testing.assert_array_equal(r.m_h, m_h)
    np.testing.assert_array_equal(cgu.stamp, cgu2.stamp)
    np.testing.assert_array_equal(cd.counters, cd2.counters)
    assert cgu.counters[0] + cgu.counters[1] == 12 * 32


def test_residual_rmsnorm_and_union():
    x = di.heavy_tail_vector(30, 64)
    y = np.linspace(-1, 1, 64)
    out = oracle.residual_rmsnorm(x, y)
    r = x.astype(np.float64) + y
    np.testing.assert_allclose(out, r / np.sqrt((r * r).mean()), rtol=1e-6)
    assert np.sqrt((out.astype(np.float64) ** 2).mean()) == pytest.approx(1.0, rel=1e-6)
    m = np.array([[1, 0, 0, 1, 0], [0, 0, 1, 1, 0], [0, 0, 0, 0, 0]], dtype=np.uint8)
    u, n = oracle.mask_union(m)
    assert u.tolist() == [1, 0, 1, 1, 0] and n == 3

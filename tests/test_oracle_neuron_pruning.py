"""Pins of the oracle's Gate pruning / Up pruning step (Sec. 3.2, Eq. 5).

Eq. 5 defines the method through pruned matrices: rows of one first-layer matrix and columns of
W^d outside the top-k neurons are zero, and the MLP is the dense one.  So the step must equal the
dense oracle (itself pinned against numpy) run on explicitly zeroed matrices; k = d_ff must be
the dense MLP; k = 1 has a closed form; a hand-worked example fixes which activation ranks."""
import numpy as np
import pytest

import oracle

F32 = 0


def _mats(rng, d_model, d_ff):
    Wg = rng.standard_normal((d_ff, d_model)).astype(np.float32)
    Wu = rng.standard_normal((d_ff, d_model)).astype(np.float32)
    Wd = rng.standard_normal((d_model, d_ff)).astype(np.float32)
    return Wg, Wu, Wd


def _wrap(Wg, Wu, Wd):
    d_ff, d_model = Wg.shape
    return (oracle.Matrix(F32, Wg, None, d_ff, d_model), oracle.Matrix(F32, Wu, None, d_ff, d_model),
            oracle.Matrix(F32, Wd, None, d_model, d_ff))


@pytest.mark.parametrize("by", ["gate", "up"])
def test_keeping_every_neuron_is_the_dense_mlp(by):
    rng = np.random.default_rng(3)
    Wg, Wu, Wd = _mats(rng, 24, 40)
    x = rng.standard_normal(24).astype(np.float32)
    r = oracle.neuron_pruned_step(*_wrap(Wg, Wu, Wd), x, 40, by)
    _, y = oracle.dense_mlp(*_wrap(Wg, Wu, Wd), x)
    assert r.m.all() and np.array_equal(r.idx, np.arange(40))
    # two binary32 roundings of intermediates (p32, h32) separate the two
    assert np.allclose(r.y, y, rtol=0, atol=1e-5 * np.abs(y).max())


@pytest.mark.parametrize("by", ["gate", "up"])
@pytest.mark.parametrize("k", [1, 5, 17, 39])
def test_equals_dense_mlp_on_the_pruned_matrices_of_eq5(by, k):
    rng = np.random.default_rng(100 + k)
    d_model, d_ff = 16, 40
    Wg, Wu, Wd = _mats(rng, d_model, d_ff)
    x = rng.standard_normal(d_model).astype(np.float32)
    r = oracle.neuron_pruned_step(*_wrap(Wg, Wu, Wd), x, k, by)
    assert int(r.m.sum()) == k and np.array_equal(np.nonzero(r.m)[0], r.idx)
    # the ranking activation, from numpy in fp64, and its k largest magnitudes (stable: lower index first)
    g, u = Wg.astype(np.float64) @ x.astype(np.float64), Wu.astype(np.float64) @ x.astype(np.float64)
    p = (g / (1.0 + np.exp(-g)) if by == "gate" else u).astype(np.float32)
    assert np.array_equal(r.p32, p)
    order = np.argsort(-np.abs(p), kind="stable")[:k]
    assert np.array_equal(np.sort(order), r.idx)
    # Eq. 5: zero the pruned rows / columns, then the dense MLP
    keep = r.m.astype(bool)
    Wg2, Wu2, Wd2 = Wg.copy(), Wu.copy(), Wd.copy()
    (Wu2 if by == "gate" else Wg2)[~keep, :] = 0.0
    Wd2[:, ~keep] = 0.0
    _, y = oracle.dense_mlp(*_wrap(Wg2, Wu2, Wd2), x)
    assert np.allclose(r.y, y, rtol=0, atol=1e-5 * max(1e-30, np.abs(y).max()))
    assert np.all(r.h32[~keep] == 0.0)


@pytest.mark.parametrize("by", ["gate", "up"])
def test_single_neuron_closed_form(by):
    rng = np.random.default_rng(9)
    Wg, Wu, Wd = _mats(rng, 8, 12)
    x = rng.standard_normal(8).astype(np.float64)
    r = oracle.neuron_pruned_step(*_wrap(Wg, Wu, Wd), x.astype(np.float32), 1, by)
    x = x.astype(np.float32).astype(np.float64)
    g, u = Wg.astype(np.float64) @ x, Wu.astype(np.float64) @ x
    a = g / (1.0 + np.exp(-g))
    j = int(np.argmax(np.abs(a if by == "gate" else u)))
    assert r.idx.tolist() == [j]
    assert np.allclose(r.y, Wd[:, j].astype(np.float64) * (a[j] * u[j]), rtol=1e-6, atol=1e-9)


def test_gate_pruning_ranks_the_activated_gate_not_the_raw_product():
    """Hand-worked: x = (1, 0).  Neuron 0 has g = -8 (silu = -0.00268...), neuron 1 has g = 1
    (silu = 0.731...), neuron 2 has g = 0.5 (silu = 0.311...).  |g| would keep neuron 0 first;
    |silu(g)| keeps neuron 1, then 2.  Up values u = (5, 2, 4)."""
    Wg = np.array([[-8.0, 0.0], [1.0, 0.0], [0.5, 0.0]], dtype=np.float32)
    Wu = np.array([[5.0, 0.0], [2.0, 0.0], [4.0, 0.0]], dtype=np.float32)
    Wd = np.array([[1.0, 10.0, 100.0]], dtype=np.float32)      # the same output row twice below (d_model = 2)
    x = np.array([1.0, 0.0], dtype=np.float32)
    mats = (oracle.Matrix(F32, Wg, None, 3, 2), oracle.Matrix(F32, Wu, None, 3, 2),
            oracle.Matrix(F32, np.vstack([Wd, Wd]), None, 2, 3))
    r1 = oracle.neuron_pruned_step(*mats, x, 1, "gate")
    assert r1.idx.tolist() == [1]
    s1 = 1.0 / (1.0 + np.exp(-1.0))
    assert np.allclose(r1.y, [10.0 * 2.0 * s1] * 2, rtol=1e-6)
    r2 = oracle.neuron_pruned_step(*mats, x, 2, "gate")
    assert r2.idx.tolist() == [1, 2]
    s2 = 0.5 / (1.0 + np.exp(-0.5))
    assert np.allclose(r2.y, [10.0 * 2.0 * s1 + 100.0 * 4.0 * s2] * 2, rtol=1e-6)
    # Up pruning on the same numbers ranks |u| = (5, 2, 4): neuron 0, then 2
    r3 = oracle.neuron_pruned_step(*mats, x, 2, "up")
    assert r3.idx.tolist() == [0, 2]
    s0 = -8.0 / (1.0 + np.exp(8.0))
    assert np.allclose(r3.y, [1.0 * 5.0 * s0 + 100.0 * 4.0 * s2] * 2, rtol=1e-6)


def test_ties_go_to_the_lower_neuron_and_bad_k_is_rejected():
    Wg = np.ones((4, 2), dtype=np.float32)
    Wu = np.ones((4, 2), dtype=np.float32)
    Wd = np.ones((2, 4), dtype=np.float32)
    x = np.array([1.0, 1.0], dtype=np.float32)
    mats = _wrap(Wg, Wu, Wd)
    assert oracle.neuron_pruned_step(*mats, x, 2, "gate").idx.tolist() == [0, 1]
    assert oracle.neuron_pruned_step(*mats, x, 3, "up").idx.tolist() == [0, 1, 2]
    with pytest.raises(ValueError):
        oracle.neuron_pruned_step(*mats, x, 5, "up")


def test_stored_formats_equal_their_decoded_values():
    """bf16 weights through the step == the same values as binary32."""
    import dip_inputs as di
    w = di.WORKLOADS["phi3_mini"].scaled(seed=4, d_model=64, d_ff=96)
    lw = di.layer_weights(w, 0)
    x = di.token_inputs(w, n_tokens=1, batch=1, d=64)[0, 0]
    bf = (oracle.Matrix(lw.wtype, lw.gate, None, 96, 64), oracle.Matrix(lw.wtype, lw.up, None, 96, 64),
          oracle.Matrix(lw.wtype, lw.down, None, 64, 96))
    f = _wrap(di.bf16_bits_to_f32(lw.gate), di.bf16_bits_to_f32(lw.up), di.bf16_bits_to_f32(lw.down))
    for by in ("gate", "up"):
        a = oracle.neuron_pruned_step(*bf, x, 24, by)
        b = oracle.neuron_pruned_step(*f, x, 24, by)
        assert np.array_equal(a.idx, b.idx) and np.array_equal(a.y, b.y)

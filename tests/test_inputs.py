"""The seeded input generators: reproducible, shaped as stated, and the temporal mixing of tokens."""
import numpy as np

import dip_inputs as di


def test_token_inputs_are_reproducible_and_unit_rms():
    w = di.WORKLOADS["phi3_mini"]
    a = di.token_inputs(w, n_tokens=5, batch=2)
    b = di.token_inputs(w, n_tokens=5, batch=2)
    assert a.dtype == np.float32 and a.shape == (5, 2, w.d_model)
    assert np.array_equal(a, b)
    assert np.allclose(np.sqrt((a.astype(np.float64) ** 2).mean(axis=2)), 1.0, atol=1e-6)
    other = di.token_inputs(w.scaled(seed=w.seed + 1), n_tokens=5, batch=2)
    assert not np.array_equal(a, other)


def test_zero_correlation_is_the_plain_draw_and_mixing_correlates_neighbours():
    w = di.WORKLOADS["phi3_medium"]
    plain = di.token_inputs(w, n_tokens=6, batch=1)
    assert np.array_equal(plain, di.token_inputs(w, n_tokens=6, batch=1, correlation=0.0))
    mixed = di.token_inputs(w, n_tokens=6, batch=1, correlation=0.9)[:, 0]
    assert np.array_equal(mixed[0], plain[0, 0])          # the first token is the first draw
    for t in range(5):
        r = np.corrcoef(mixed[t], mixed[t + 1])[0, 1]
        assert 0.8 < r < 0.97
    far = np.corrcoef(plain[0, 0], plain[1, 0])[0, 1]
    assert abs(far) < 0.1


def test_keep_count_and_capacity_conventions():
    assert di.keep_count(0.25, 17920) == 4480 and di.keep_count(0.1, 5120) == 512
    assert di.keep_count(1e-9, 64) == 1 and di.keep_count(1.0, 64) == 64
    assert di.cache_capacity(0.4, 4096) == 1638 and di.cache_capacity(0.5, 5120) == 2560

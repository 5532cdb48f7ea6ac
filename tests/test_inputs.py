"""The seeded input generators: determinism and the structure the workloads rely on."""
import numpy as np

from paper_1902_01981_b200 import inputs


def test_generators_are_deterministic():
    a = inputs.partition_gradients(5, 100, seed=3, std=0.5)
    b = inputs.partition_gradients(5, 100, seed=3, std=0.5)
    assert a.dtype == np.float32 and np.array_equal(a, b)
    assert not np.array_equal(a, inputs.partition_gradients(5, 100, seed=4, std=0.5))
    g = inputs.integer_gradients(4, 1000, seed=1, bound=7)
    assert g.dtype == np.int32 and g.min() >= -7 and g.max() <= 7


def test_straggler_masks_respect_the_tolerance():
    n, L, s = 5, 2, 2
    m = inputs.straggler_masks(n, L, s, 200, seed=9)
    assert m.shape == (200, inputs.group_count(n, L)) and m.dtype == np.uint32
    pop = np.array([[bin(int(x)).count("1") for x in row] for row in m])
    assert pop.max() <= s and (m < (1 << n)).all()
    assert set(np.unique(pop)) == {0, 1, 2}          # every count occurs
    exact = inputs.straggler_masks(n, L, s, 50, seed=9, exactly_s=True)
    assert all(bin(int(x)).count("1") == s for x in exact.reshape(-1))


def test_linreg_labels_follow_the_true_model():
    X, y, w_star = inputs.linreg_partitions(3, 40, 16, seed=2, x_std=1.0, noise_std=0.0)
    for p in range(3):
        assert np.allclose(y[p], X[p].astype(np.float64) @ w_star.astype(np.float64), rtol=1e-6, atol=1e-6)


def test_logistic_labels_are_binary():
    _, y, _ = inputs.logistic_partitions(2, 500, 8, seed=5)
    assert set(np.unique(y)) == {0.0, 1.0}


def test_replicate_into_slots_is_a_gather():
    G = inputs.partition_gradients(6, 10, seed=0)
    slots = inputs.replicate_into_slots(G, np.array([[0, 5], [3, 3]]))
    assert slots.shape == (2, 2, 10) and np.array_equal(slots[0, 1], G[5]) and np.array_equal(slots[1, 0], G[3])


def test_tf32_representable():
    x = inputs.partition_gradients(4, 1000, 3)
    r = inputs.tf32_representable(x)
    assert r.dtype == np.float32 and (r.view(np.uint32) & 0x1FFF).max() == 0
    assert np.abs(r - x).max() <= np.abs(x).max() * 2.0 ** -11      # half a unit in the 10th mantissa bit
    assert np.array_equal(inputs.tf32_representable(r), r)          # idempotent
    assert np.array_equal(inputs.tf32_representable(np.array([1.0, -0.5, 0.0], np.float32)),
                          np.array([1.0, -0.5, 0.0], np.float32))


def test_model_matrix_spreads_around_one_start():
    W = inputs.model_matrix(8, 4096, seed=1, spread=0.1)
    assert W.shape == (8, 4096) and W.dtype == np.float32
    assert 0.05 < np.std(W - W.mean(axis=0)) < 0.15


def test_shifted_exponential_times_have_the_shift_and_the_mean():
    t = inputs.shifted_exponential_times(20000, load_points=4.0, a=2.0, mu=0.5, seed=1)
    assert t.min() >= 8.0                              # shift a * d_i
    assert abs(t.mean() - (8.0 + 4.0 / 0.5)) < 0.3     # mean a d_i + d_i / mu

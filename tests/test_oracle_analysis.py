"""The analysis helpers (Eq. 2, Eq. 5, the token-order comparison of Sec. 3.2) against what the
mathematics fixes, and the qualitative finding on values with token-level structure."""
import numpy as np

from oracle import analysis as A
from oracle import codecs as C


def test_error_decomposition_is_an_identity():
    rng = np.random.default_rng(0)
    p = rng.random((5, 40)); p /= p.sum(axis=1, keepdims=True)
    v = rng.normal(size=(40, 8))
    p_q = C.e4m3_decode(C.e4m3_encode((p * 256).astype(np.float32))) / 256
    v_q = C.e4m3_decode(C.e4m3_encode(v.astype(np.float32)))
    total, first, second = A.error_decomposition(p, p_q, v, v_q)
    assert np.abs(total - (first + second)).max() < 1e-12


def test_energy_share_is_one_for_constant_blocks_and_zero_for_centred_ones():
    const = np.repeat(np.arange(1, 4, dtype=np.float64)[:, None], 128, axis=0).reshape(3 * 128, 1) * np.ones((1, 4))
    assert abs(A.energy_share_removed(const, A.sequence_order(384)) - 1.0) < 1e-12
    x = np.tile(np.array([[1.0], [-1.0]]), (64, 4))
    assert A.energy_share_removed(x, A.sequence_order(128)) < 1e-12


def test_static_cube_order_is_a_permutation_of_bricks():
    order = A.static_cube_order((4, 4, 32))
    assert sorted(order.tolist()) == list(range(512))
    first = order[:128]                                  # the first brick: t < 4, y < 2, x < 16
    t, y, x = first // 128, (first // 32) % 4, first % 32
    assert t.max() == 3 and y.max() == 1 and x.max() == 15


def test_grouping_by_value_lowers_the_value_error_where_rotation_does_not():
    """Values = a few token-level components (which token carries which one is scattered over the
    sequence) + noise: sorting by k-means lets the block mean remove the shared component, a
    Hadamard rotation of the channels leaves the error where it was (Sec. 3.2, token-order table)."""
    rng = np.random.default_rng(1)
    n, d, k = 2048, 32, 8
    centres = rng.normal(size=(k, d)) * 3.0
    which = rng.integers(0, k, size=n)
    v = C.bf16_round((centres[which] + 0.3 * rng.normal(size=(n, d))).astype(np.float32)).astype(np.float64)
    seq, km = A.sequence_order(n), A.kmeans_order(v, k=k, iters=4)
    e_seq, e_had, e_km = A.value_rmse(v, seq), A.value_rmse(v, seq, hadamard=True), A.value_rmse(v, km)
    assert e_km < 0.5 * e_seq
    assert 0.5 * e_seq < e_had < 2.0 * e_seq
    assert A.energy_share_removed(v, km) > A.energy_share_removed(v, seq) + 0.3
    rows = A.report(v, (8, 16, 16), k=k)
    assert [r[0] for r in rows] == ["sequence", "Hadamard on V", "static cube 4x2x16", "k-means"]

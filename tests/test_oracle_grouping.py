"""Pins of the grouping oracle (Sec. 3.2 "Value-guided permutation") against what the
mathematics fixes: brute-force nearest-centroid search, recovery of separated clusters, the
monotone k-means objective, the empty-cluster rule, and the definition of a stable sort."""
import numpy as np

from oracle import grouping as G


def _blobs(rng, k, per, d, spread=0.05):
    centers = rng.normal(size=(k, d)) * 4.0
    x = np.concatenate([centers[j] + spread * rng.normal(size=(per, d)) for j in range(k)])
    truth = np.repeat(np.arange(k), per)
    p = rng.permutation(x.shape[0])
    return x[p], truth[p], centers


def test_assign_is_the_nearest_centroid_by_brute_force():
    rng = np.random.default_rng(0)
    x, c = rng.normal(size=(37, 5)), rng.normal(size=(6, 5))
    labels, margin = G.assign(x, c)
    for t in range(37):
        best, arg = None, None
        for j in range(6):
            dist = sum((x[t, i] - c[j, i]) ** 2 for i in range(5))
            if best is None or dist < best:        # strict: ties keep the lower index
                best, arg = dist, j
        assert labels[t] == arg
    assert (margin >= 0).all()


def test_ties_go_to_the_lower_index():
    x = np.array([[0.0, 0.0]])
    c = np.array([[1.0, 0.0], [-1.0, 0.0], [0.0, 1.0]])
    assert G.assign(x, c)[0][0] == 0


def test_separated_clusters_are_recovered_and_sorted_into_runs():
    rng = np.random.default_rng(1)
    x, truth, centers = _blobs(rng, 8, 50, 16)
    # start from one member of each true cluster so that no cluster is lost to a bad start
    start = np.stack([x[np.nonzero(truth == j)[0][0]] for j in range(8)])
    labels, c, _, _ = G.kmeans(x, 8, 3, centroids=start)
    assert (labels == truth).all()
    assert np.abs(c - centers).max() < 0.05
    pi = G.stable_argsort(labels)
    assert sorted(pi.tolist()) == list(range(400))
    assert (np.diff(truth[pi]) >= 0).all()          # every cluster one contiguous run


def test_objective_never_increases():
    rng = np.random.default_rng(2)
    x = rng.normal(size=(500, 8))
    _, _, _, obj = G.kmeans(x, 16, 6)
    assert all(b <= a * (1 + 1e-12) for a, b in zip(obj, obj[1:]))


def test_empty_cluster_keeps_its_centroid_and_update_is_the_mean():
    x = np.array([[0.0], [1.0], [10.0], [11.0]])
    c0 = np.array([[0.0], [10.0], [100.0]])
    labels, _ = G.assign(x, c0)
    c1 = G.update(x, labels, c0)
    assert labels.tolist() == [0, 0, 1, 1]
    assert c1[:, 0].tolist() == [0.5, 10.5, 100.0]


def test_initial_centroids_are_every_n_over_k_th_row():
    x = np.arange(20, dtype=np.float64).reshape(10, 2)
    assert G.initial_centroids(x, 3)[:, 0].tolist() == [0.0, 6.0, 12.0]   # rows 0, 3, 6


def test_stable_argsort_definition():
    labels = np.array([2, 0, 1, 0, 2, 1, 0])
    pi = G.stable_argsort(labels)
    assert pi.tolist() == [1, 3, 6, 2, 5, 0, 4]
    assert pi.tolist() == np.argsort(labels, kind="stable").tolist()

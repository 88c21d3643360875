"""Value-guided permutation (Sec. 3.2) -- CPU oracle, TEST INFRASTRUCTURE.

Per (batch, head): a k-means over the value tokens gives a label z_t per token, and
pi = argsort(z) (Eq. 3) puts every cluster into one contiguous run of K/V rows.  The paper
says "online k-means", warm-started from the previous step's centroids, plain (unbalanced);
it fixes neither k, nor the initialisation, nor the iteration count.  Reading taken by this
build: Lloyd iterations (assign every token to the nearest centroid in squared Euclidean
distance, ties to the lower index; then move every centroid to the mean of its members, an
empty cluster keeping its centroid), centroids started at rows 0, N//k, 2(N//k), ... unless
given, labels of the LAST assignment, argsort stable (token order kept inside a cluster).
All arithmetic in fp64 on the bf16-exact inputs.  parity unpinned for k / init / iterations.
"""
import numpy as np


def assign(x, c):
    """Nearest centroid per row of x (ties -> lower index) and the margin to the runner-up.

    The distance is written out as |x - c|^2 (no expansion), row by row."""
    x = np.asarray(x, dtype=np.float64)
    c = np.asarray(c, dtype=np.float64)
    labels = np.empty(x.shape[0], dtype=np.int64)
    margin = np.empty(x.shape[0], dtype=np.float64)
    for lo in range(0, x.shape[0], 4096):
        diff = x[lo:lo + 4096, None, :] - c[None, :, :]
        d2 = (diff * diff).sum(axis=2)
        lab = d2.argmin(axis=1)                      # first minimum = lower index on ties
        labels[lo:lo + 4096] = lab
        if c.shape[0] > 1:
            part = np.partition(d2, 1, axis=1)
            margin[lo:lo + 4096] = part[:, 1] - part[:, 0]
        else:
            margin[lo:lo + 4096] = np.inf
    return labels, margin


def update(x, labels, c):
    """Centroid <- mean of its members; an empty cluster keeps its centroid."""
    x = np.asarray(x, dtype=np.float64)
    out = np.array(c, dtype=np.float64, copy=True)
    for j in range(out.shape[0]):
        members = x[labels == j]
        if members.shape[0] > 0:
            out[j] = members.sum(axis=0) / members.shape[0]
    return out


def initial_centroids(x, k):
    step = max(x.shape[0] // k, 1)
    return np.asarray(x, dtype=np.float64)[::step][:k].copy()


def kmeans(x, k, iters, centroids=None):
    """Returns (labels of the last assignment, centroids after the last update, margins,
    objective before each assignment's update)."""
    x = np.asarray(x, dtype=np.float64)
    c = initial_centroids(x, k) if centroids is None else np.asarray(centroids, dtype=np.float64).copy()
    labels = margin = None
    objective = []
    for _ in range(iters):
        labels, margin = assign(x, c)
        objective.append(float(((x - c[labels]) ** 2).sum()))
        c = update(x, labels, c)
    return labels, c, margin, objective


def stable_argsort(labels):
    """pi with labels[pi] non-decreasing and token order kept among equal labels (Eq. 3)."""
    labels = np.asarray(labels)
    order = []
    for j in range(int(labels.max()) + 1 if labels.size else 0):
        order.extend(np.nonzero(labels == j)[0].tolist())
    return np.asarray(order, dtype=np.int64)

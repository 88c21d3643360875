"""A plain PyTorch k-means permutation for the harness (tests and `bench.py --perm kmeans`).

Not part of the product and not the oracle: it is an independent, library-level way to get a
value-guided token permutation (Sec. 3.2 "Value-guided permutation") to feed BOTH the CUDA
path and the oracle with, and a comparison point for `vc_group`.  The library's own producer
of the permutation is `vc_group`; its oracle is `oracle/grouping.py`.
"""
import torch


def kmeans_perm(v, k=64, iters=4, centroids=None):
    """Token grouping for one head: Lloyd iterations on the fp32 value rows, then a stable
    argsort of the labels (Sec. 3.2 "Value-guided permutation").  The paper fixes neither
    k nor the initialisation; this harness takes k = 64, centroids started at every
    (N // k)-th token (or warm-started from `centroids`), squared Euclidean distance, an
    empty cluster keeping its centroid.  Returns (perm int32 [N], centroids [k, d]).
    """
    x = v.float()
    N = x.shape[0]
    k = min(k, N)
    c = x[:: max(N // k, 1)][:k].clone() if centroids is None else centroids.clone()
    labels = None
    for _ in range(iters):
        d2 = (x * x).sum(1, keepdim=True) - 2.0 * (x @ c.T) + (c * c).sum(1)[None, :]
        labels = d2.argmin(dim=1)
        sums = torch.zeros_like(c).index_add_(0, labels, x)
        cnt = torch.zeros(c.shape[0], device=x.device).index_add_(0, labels, torch.ones(N, device=x.device))
        c = torch.where(cnt[:, None] > 0, sums / cnt.clamp(min=1)[:, None], c)
    perm = torch.sort(labels, stable=True).indices
    return perm.to(torch.int32), c


def kmeans_perm_all(v, k=64, iters=4):
    """[B, H, N, d] -> int32 [B, H, N]."""
    B, H, N, _ = v.shape
    out = torch.empty(B, H, N, dtype=torch.int32, device=v.device)
    for b in range(B):
        for h in range(H):
            out[b, h], _ = kmeans_perm(v[b, h], k, iters)
    return out

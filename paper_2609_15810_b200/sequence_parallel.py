"""Head-sharded VC-Attention for callers whose activations are sharded along the sequence.

Every (batch, head) is independent through the whole path (the permutation, the K mean, the
value scales and the block means are per head, Sec. 3.2 and App. B), so the path itself has no
exchange step: with G GPUs each one runs H/G heads.  A caller that holds the SEQUENCE sharded
(each rank a contiguous slice of N/G tokens of every head) needs one all-to-all in front
(sequence shards -> head shards, for Q, K and V) and one behind (for O).  That exchange is
plain NCCL through torch.distributed; nothing inside the kernels crosses GPUs.

    q, k, v : [B, H, N/G, d] bf16 on this rank (tokens rank*N/G ... of every head)
    returns : [B, H, N/G, d] bf16, the same slice of the output

One process per GPU, torch.distributed initialised by the caller.
"""
import torch
import torch.distributed as dist

from .binding import Params, alloc_buffers, vc_attn, vc_group, vc_group_workspace_bytes, vc_poll_status


def _world(group):
    return dist.get_world_size(group) if dist.is_initialized() else 1


def _all_to_all(send, group):
    """send: [G, ...] contiguous, slab r goes to rank r; returns [G, ...] with slab r from rank r."""
    if _world(group) == 1:
        return send
    recv = torch.empty_like(send)
    dist.all_to_all_single(recv, send, group=group)
    return recv


def seq_to_head_shard(x, group=None):
    """[B, H, N/G, d] (my token slice of every head) -> [B, H/G, N, d] (every token of my heads).

    Rank r receives heads r*H/G ... (r+1)*H/G - 1; token slices are concatenated in rank order."""
    G = _world(group)
    B, H, n, d = x.shape
    if H % G:
        raise ValueError(f"H = {H} is not divisible by the number of ranks {G}")
    send = x.reshape(B, G, H // G, n, d).permute(1, 0, 2, 3, 4).contiguous()      # [G][B, H/G, n, d]
    recv = _all_to_all(send, group)                                               # slab r: rank r's tokens
    return recv.permute(1, 2, 0, 3, 4).reshape(B, H // G, G * n, d)


def head_to_seq_shard(o, group=None):
    """[B, H/G, N, d] (every token of my heads) -> [B, H, N/G, d] (my token slice of every head)."""
    G = _world(group)
    B, h, N, d = o.shape
    if N % G:
        raise ValueError(f"N = {N} is not divisible by the number of ranks {G}")
    n = N // G
    send = o.reshape(B, h, G, n, d).permute(2, 0, 1, 3, 4).contiguous()           # [G][B, H/G, n, d]
    recv = _all_to_all(send, group)                                               # slab r: rank r's heads
    return recv.permute(1, 0, 2, 3, 4).reshape(B, G * h, n, d)


def vc_attn_sequence_parallel(q, k, v, grid, bits=8, group=None, group_k=0, group_iters=4, **params):
    """VC-Attention over sequence-sharded Q, K, V.  `grid` is the (T, H, W) token grid of the FULL
    sequence; `group_k` > 0 builds the token-group permutation of the local heads with vc_group
    (cold start), 0 runs without permutation; other keyword arguments go to Params.make."""
    qh, kh, vh = (seq_to_head_shard(t, group) for t in (q, k, v))
    B, h, N, d = qh.shape
    p = Params.make(B, h, N, d, grid, bits=bits, **params)
    perm = None
    if group_k > 0:
        gwork = torch.empty(vc_group_workspace_bytes(p), dtype=torch.uint8, device=qh.device)
        centroids = torch.zeros(B, h, group_k, d, dtype=torch.float32, device=qh.device)
        perm = torch.empty(B, h, N, dtype=torch.int32, device=qh.device)
        vc_group(p, vh, group_k, group_iters, False, centroids, perm, gwork)
    quant, work = alloc_buffers(p)
    o = torch.empty(B, h, N, d, dtype=torch.bfloat16, device=qh.device)
    vc_attn(p, qh, kh, vh, perm, o, quant, work)
    vc_poll_status(work)
    return head_to_seq_shard(o, group)

"""Plumbing for the one-worker-per-GPU form: make every worker's theta buffers addressable in
every process.  PyTorch does the work (its CUDA-IPC tensor sharing and a torch.distributed group
for passing the handles around); nothing of the method is computed here."""
from __future__ import annotations

import torch.distributed as dist
from torch.multiprocessing.reductions import reduce_tensor


def exchange_buffers(own: list, group=None) -> list:
    """``own`` = this rank's CUDA tensors (e.g. its two theta buffers).  Returns ``views`` with
    ``views[r][i]`` a tensor that aliases tensor i of rank r (rank's own entries are the originals).
    The other ranks' memory is mapped through CUDA IPC, so it works for processes on the same GPU
    and, with peer access, on different GPUs of one node.  Keep the returned tensors alive for as
    long as the addresses are in use; the owners must keep their originals alive too."""
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    packed = [reduce_tensor(t) for t in own]
    gathered = [None] * world
    dist.all_gather_object(gathered, packed, group=group)
    views = []
    for r in range(world):
        if r == rank:
            views.append(list(own))
        else:
            views.append([fn(*args) for fn, args in gathered[r]])
    dist.barrier(group=group)          # everybody has opened everybody's handles
    return views

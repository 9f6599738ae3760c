"""Multi-GPU plumbing: one process per GPU, ciphertext-index shards, no data-path collective.

Every ciphertext index is independent through the whole round (encode, encrypt, neighbour
sums, shares, combine, decode all act per index across parties) and all key material is
re-derived on each GPU from (parameters, seed), so ranks never exchange polynomials.  The
only communication is the rendezvous, the barriers around the timed region and the
max-reduction of the measured time.
"""
import os

import torch
import torch.distributed as dist


def env_world():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("LOCAL_RANK", "0")),
            int(os.environ.get("WORLD_SIZE", "1")))


def init(backend=None):
    """Joins the process group described by the torchrun environment (no-op for one process)."""
    rank, local_rank, world = env_world()
    if world > 1 and not dist.is_initialized():
        if backend is None:
            backend = "nccl" if torch.cuda.is_available() else "gloo"
        if backend == "nccl":
            torch.cuda.set_device(local_rank)
        dist.init_process_group(backend)
    return rank, local_rank, world


def barrier(device=None):
    if dist.is_initialized():
        dist.barrier()
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)


def max_over_ranks(value, device=None):
    """Max of a Python float over all ranks (the slowest rank defines the step time)."""
    if not dist.is_initialized():
        return float(value)
    t = torch.tensor([float(value)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def gather_to_rank0(tensor_cpu):
    """Concatenates per-rank CPU tensors along dim 1 (ciphertext index) on rank 0."""
    if not dist.is_initialized():
        return tensor_cpu
    world = dist.get_world_size()
    parts = [torch.empty_like(tensor_cpu) for _ in range(world)] if dist.get_rank() == 0 else None
    dist.gather(tensor_cpu, parts, dst=0)
    return torch.cat(parts, dim=1) if parts is not None else None


def finish():
    if dist.is_initialized():
        dist.destroy_process_group()

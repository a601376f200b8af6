"""Replica bookkeeping for runs on several GPUs.

The decode-attention path shards by (sequence, layer, KV head) with no exchange step: every team
record, Philox sub-stream and output belongs to one (sequence, KV head) (Algorithm 1 is stated per
query head; Section "method" builds teams separately for each layer and KV head). Several GPUs
therefore run independent replicas: each rank owns its own sequences and no collective touches the
data path. The process group is used for two things only, both here: the barrier that brackets a
timed region and the maximum over ranks of the device-measured time.

Nothing in this module needs a GPU; the multi-process CPU tests run it over the gloo backend.
"""
import os
from typing import Optional

import torch
import torch.distributed as dist


def env_rank_world():
    """(rank, world size, local rank) as torchrun exports them; (0, 1, 0) when launched directly."""
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def init_replicas(backend: str, device: Optional[torch.device] = None) -> int:
    """Join the process group named by the environment (MASTER_ADDR/MASTER_PORT/RANK/WORLD_SIZE).
    Returns the world size; does nothing for a single process."""
    _, world, _ = env_rank_world()
    if world > 1 and not dist.is_initialized():
        if backend == "nccl":
            dist.init_process_group("nccl", device_id=device)
        else:
            dist.init_process_group(backend)
    return world


def replica_seed(base_seed: int, rank: int) -> int:
    """Seed of a rank's synthetic sequences and of its sampling stream: replicas are independent."""
    return int(base_seed) + int(rank)


def barrier(device: Optional[torch.device] = None) -> None:
    """Device synchronisation, then a barrier over the ranks, then device synchronisation again."""
    if device is not None and device.type == "cuda":
        torch.cuda.synchronize(device)
    if dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()
        if device is not None and device.type == "cuda":
            torch.cuda.synchronize(device)


def max_over_ranks(ms: float, device: Optional[torch.device] = None) -> float:
    """Largest of the ranks' device-measured times: the job is as slow as its slowest replica."""
    if not (dist.is_initialized() and dist.get_world_size() > 1):
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device if device is not None else torch.device("cpu"))
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def us_per_layer_step(ms: float, steps: int, layers: int, world: int) -> float:
    """Whole-job microseconds per layer-step: every rank ran steps * layers layer-steps in `ms`."""
    return 1e3 * ms / (steps * layers * world)

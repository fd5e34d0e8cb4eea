"""Host-side logic of multi-GPU runs.  The calibration path has no exchange step between
GPUs: every rank calibrates its own rotation site (an independent seeded problem), so N GPUs
are N replicas and the only collective is the max over ranks of the measured times.

One process per GPU.  A program either finds its rank in the environment (an external launcher
such as torch.distributed.run set RANK / LOCAL_RANK / WORLD_SIZE / MASTER_*) or starts its own
ranks on this node with `launch`."""
from __future__ import annotations

import os
import socket
import subprocess
import sys
from dataclasses import replace


def workload_for_rank(w, rank: int):
    """The problem rank `rank` calibrates: same recipe, its own seed (rank 0 keeps the base seed)."""
    return replace(w, seed=w.seed + rank)


def launched_externally() -> bool:
    """True when a launcher already put this process's rank into the environment."""
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch(world: int, argv, timeout=None, capture_rank0: bool = False):
    """Start `world` ranks of `python argv...` on this node and wait for them.

    Rank r gets RANK = LOCAL_RANK = r, WORLD_SIZE = world, MASTER_ADDR = 127.0.0.1 and a free
    MASTER_PORT.  Rank 0 writes to this process's stdout (or, with capture_rank0, to a pipe whose
    text is returned); the other ranks' stdout is discarded, everyone's stderr is inherited.
    Returns (exit codes, rank 0's stdout or None).  If a rank fails the others are terminated."""
    port = free_port()
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        out = (subprocess.PIPE if capture_rank0 else None) if r == 0 else subprocess.DEVNULL
        procs.append(subprocess.Popen([sys.executable] + list(argv), env=env, stdout=out, text=True))
    text = None
    try:
        if capture_rank0:
            text, _ = procs[0].communicate(timeout=timeout)
        codes = [p.wait(timeout=timeout) for p in procs]
    except BaseException:
        for p in procs:
            if p.poll() is None:
                p.terminate()
        raise
    return codes, text


def init_process_group(backend: str):
    """(rank, local_rank, world) from the environment; joins the process group when world > 1."""
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        import torch
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        kw = {}
        if backend == "nccl":
            kw["device_id"] = torch.device("cuda", local_rank)
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, local_rank, world


def barrier():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.barrier()


def shutdown():
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()


def max_over_ranks(values, device="cpu"):
    """Element-wise max of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units all ranks processed divided by the slowest rank's time (weak scaling)."""
    return world * units_per_rank / (ms_max * 1e-3)


def headline(metric: str, unit: str, units_per_rank: float, world: int, ms_local: float, device="cpu") -> dict:
    """The rank-independent part of a benchmark line: every rank passes its own time for
    `units_per_rank` units; the result (identical on all ranks) carries the whole-job rate over the
    slowest rank's time."""
    (ms,) = max_over_ranks([ms_local], device=device)
    return {"metric": metric, "value": whole_job_rate(units_per_rank, world, ms), "unit": unit, "n_gpus": world,
            "ms_per_step": ms / units_per_rank, "scaling": "weak", "parallelism": "replicas x%d" % world}

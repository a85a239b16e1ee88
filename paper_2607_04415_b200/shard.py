"""Query sharding for multi-GPU runs: queries are independent, so rank r of `world` takes a
contiguous slice and owns a private page cache, request ring and proxy.  No data-path
collective exists; results are gathered only if the caller wants them in one place."""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_range(nq: int, rank: int, world: int):
    """Half-open [begin, end) of the queries rank `rank` searches (sizes differ by at most 1)."""
    base, rem = divmod(nq, world)
    begin = rank * base + min(rank, rem)
    return begin, begin + base + (1 if rank < rem else 0)


def gather_results(local: torch.Tensor, nq: int):
    """All-gather per-rank result rows (ragged along dim 0) into the global [nq, ...] order."""
    world, rank = dist.get_world_size(), dist.get_rank()
    sizes = [shard_range(nq, r, world)[1] - shard_range(nq, r, world)[0] for r in range(world)]
    pad = max(sizes)
    buf = torch.zeros((pad,) + tuple(local.shape[1:]), dtype=local.dtype, device=local.device)
    buf[: local.shape[0]] = local
    parts = [torch.empty_like(buf) for _ in range(world)]
    dist.all_gather(parts, buf)
    return torch.cat([p[:s] for p, s in zip(parts, sizes)], 0)


def free_port() -> int:
    """A TCP port that is free on 127.0.0.1 right now (for the rendezvous of a local launch)."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n_ranks: int, script: str, argv, env=None, timeout=None) -> int:
    """Run `script argv...` as n_ranks processes of one node, one per GPU, the way a launcher
    would: `python -m torch.distributed.run --nnodes=1 --nproc-per-node n --master-addr 127.0.0.1
    --master-port <free port> script argv...`, so that every child finds RANK, LOCAL_RANK,
    WORLD_SIZE and MASTER_* in its environment.  Returns the launcher's exit code (non-zero if
    any rank failed).  The children share nothing on the device: no collective is on the data path."""
    import os
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n_ranks)}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script] + list(argv)
    e = dict(os.environ if env is None else env)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):      # the launcher sets these for its children
        e.pop(k, None)
    return subprocess.run(cmd, env=e, timeout=timeout).returncode


def parse_cpulist(text: str):
    """'0-3,8,10-11' -> {0, 1, 2, 3, 8, 10, 11} (the format of sysfs cpulist files)."""
    cpus = set()
    for part in text.strip().split(","):
        if not part:
            continue
        lo, _, hi = part.partition("-")
        cpus.update(range(int(lo), int(hi or lo) + 1))
    return cpus


def bind_to_gpu_cpus(pci_bus: str, sysfs_root: str = "/sys") -> bool:
    """Restrict this process to the CPUs next to a GPU (sysfs `local_cpulist` of its PCI device), so
    that the page store a rank allocates and pins afterwards, its proxy thread and the words that
    thread polls sit on the GPU's own socket: with one rank per GPU on a two-socket host, a page
    store on the far socket makes every page pull cross the socket interconnect.  Best effort: it
    does nothing (and returns False) when the file is missing, names no CPU this process may use,
    or names all of them.  `pci_bus` is 'dddd:bb:dd.f', lower case."""
    import os
    try:
        with open(os.path.join(sysfs_root, "bus/pci/devices", pci_bus, "local_cpulist")) as fh:
            local = parse_cpulist(fh.read())
        allowed = os.sched_getaffinity(0)
        want = local & allowed
        if not want or want == allowed:
            return False
        os.sched_setaffinity(0, want)
        return True
    except (OSError, ValueError):
        return False

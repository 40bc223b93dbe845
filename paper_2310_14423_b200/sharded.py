"""Algorithm 2 with the K workers sharded over several processes (one GPU each).

This is the paper's own layout -- one worker (here: a block of workers) per GPU, parameters averaged by an
All-Reduce at the end of each round -- and the only exchange step on the path: local steps need no
communication.  Per round each process
    1. takes H - 1 local steps on its rows                              (qsr_local_step)
    2. takes the last step and sums its rows' new parameters into a [P] buffer, in one launch that does not even
       write the parameter rows                                         (qsr_local_step_partial)
    3. all-reduces that buffer (SUM) over processes                     (torch.distributed: NCCL over NVLink)
    4. divides by the global worker count and writes every local row    (qsr_sync_finish)
The round length comes from the host schedule, which depends only on t, so every process computes the same H
without talking to the others.  Noise is addressed by the *global* worker index (worker_offset + local row).

The functions here only sequence calls; the arithmetic is the engine's.  `engine` is a binding.Context in the
product; any object with the same methods can stand in for it (the CPU tests drive this loop over gloo).
"""
from __future__ import annotations

from typing import List, Tuple


def shard(K_total: int, world_size: int, rank: int) -> Tuple[int, int]:
    """(number of workers held by `rank`, global index of its first worker): contiguous blocks, sizes differ by <= 1."""
    if not (0 <= rank < world_size) or K_total < world_size:
        raise ValueError("need at least one worker per process")
    base, rem = divmod(K_total, world_size)
    k_local = base + (1 if rank < rem else 0)
    offset = rank * base + min(rank, rem)
    return k_local, offset


def run_rounds(engine, sums, K_total: int, t_begin: int, t_end: int, all_reduce) -> List[Tuple[int, int]]:
    """Rounds that start in [t_begin, t_end), each run to its end.  `sums` is the [qsr_sync_sum_floats] buffer the
    engine writes its partial sums to; `all_reduce(sums)` must SUM it in place over all processes.
    Returns [(round start, round length)]."""
    rounds = []
    t = int(t_begin)
    while t < t_end:
        H = engine.qsr_round_length(t)
        for h in range(H - 1):
            engine.qsr_local_step(t + h)
        engine.qsr_local_step_partial(t + H - 1, sums)    # last step + this process's row sums, one launch
        all_reduce(sums)
        engine.qsr_sync_finish(sums, K_total, t + H)
        rounds.append((t, H))
        t += H
    return rounds

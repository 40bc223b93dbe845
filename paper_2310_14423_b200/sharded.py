"""Algorithm 2 as a sequence of library calls, on one GPU or with the K workers sharded over several processes.

Sharding is the paper's own layout -- one worker (here: a block of workers) per GPU, parameters averaged by an
All-Reduce at the end of each round -- and the only exchange step on the path: local steps need no
communication.  Per round each process
    1. takes H - 1 local steps on its rows                              (qsr_local_step)
    2. takes the last step and sums its rows' new parameters into a [P] buffer, in one launch that does not even
       write the parameter rows                                         (qsr_local_step_partial)
    3. all-reduces that buffer (SUM) over processes                     (torch.distributed: NCCL over NVLink)
    4. divides by the global worker count and writes every local row    (qsr_sync_finish)
On one GPU steps 2-4 are a single launch (qsr_local_step_sync).
The round length comes from the host schedule, which depends only on t, so every process computes the same H
without talking to the others.  Noise is addressed by the *global* worker index (worker_offset + local row).

The functions here only sequence calls; the arithmetic is the engine's.  `engine` is a binding.Context in the
product; any object with the same methods can stand in for it (the CPU tests drive this loop over gloo).  The
benchmark times exactly this loop, so what the multi-process tests cover is what a multi-GPU run executes.
"""
from __future__ import annotations

from typing import Callable, List, NamedTuple, Optional, Tuple


class Exchange(NamedTuple):
    """What a sharded round end needs: the [qsr_sync_sum_floats] buffer the engine writes its partial sums to (in
    state mode AVERAGE the sums of state1 / state2 follow those of the parameters, each region P rounded up to 4
    floats), the global worker count, and a callable that SUMs the buffer in place over all processes."""
    sums: object
    K_total: int
    all_reduce: Callable[[object], None]


def shard(K_total: int, world_size: int, rank: int) -> Tuple[int, int]:
    """(number of workers held by `rank`, global index of its first worker): contiguous blocks, sizes differ by <= 1."""
    if not (0 <= rank < world_size) or K_total < world_size:
        raise ValueError("need at least one worker per process")
    base, rem = divmod(K_total, world_size)
    k_local = base + (1 if rank < rem else 0)
    offset = rank * base + min(rank, rem)
    return k_local, offset


def run_steps(engine, t_begin: int, t_end: int, exchange: Optional[Exchange] = None,
              on_launch: Optional[Callable[[str, int], None]] = None, whole_rounds: bool = False) -> List[Tuple[int, int]]:
    """Global steps [t_begin, t_end) of Algorithm 2; t_begin must be the first step of a round.

    A round that ends inside the window ends with its synchronization: on one GPU (`exchange` is None) the last step
    carries the averaging itself; otherwise the last step writes this process's row sums, `exchange.all_reduce` sums
    them over processes and the finish launch writes the global mean to every local row.  With `whole_rounds` the
    last round is run to its end even if that lies beyond t_end; without it the window may stop inside a round.
    `on_launch(kind, t)` is called after the launches of step t have been enqueued, kind "step" for a plain local
    step and "sync" for a step that also ends its round (a place to record an event).
    Returns [(round start, round length)] of the rounds completed."""
    rounds = []
    t = int(t_begin)
    while t < t_end:
        H = engine.qsr_round_length(t)
        last = t + H - 1
        stop = t + H if whole_rounds else min(t + H, int(t_end))
        for u in range(t, min(stop, last)):
            engine.qsr_local_step(u)
            if on_launch:
                on_launch("step", u)
        if stop == t + H:
            if exchange is None:
                engine.qsr_local_step_sync(last, t + H)           # last step and averaging, one launch
            else:
                engine.qsr_local_step_partial(last, exchange.sums)    # last step + this process's row sums
                exchange.all_reduce(exchange.sums)
                engine.qsr_sync_finish(exchange.sums, exchange.K_total, t + H)
            if on_launch:
                on_launch("sync", last)
            rounds.append((t, H))
        t += H
    return rounds


def run_rounds(engine, sums, K_total: int, t_begin: int, t_end: int, all_reduce) -> List[Tuple[int, int]]:
    """Sharded rounds that start in [t_begin, t_end), each run to its end.  `sums` is the [qsr_sync_sum_floats] buffer
    the engine writes its partial sums to; `all_reduce(sums)` must SUM it in place over all processes.
    Returns [(round start, round length)]."""
    return run_steps(engine, t_begin, t_end, Exchange(sums, K_total, all_reduce), whole_rounds=True)

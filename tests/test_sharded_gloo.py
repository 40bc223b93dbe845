"""The replica-sharded round loop on CPU: two (and three) gloo ranks, each holding a block of workers.

The loop under test is the product's (`sharded.run_rounds`, i.e. `sharded.run_steps`, round lengths from the library's
host schedule); the arithmetic of each rank is supplied by the CPU oracle standing in for the CUDA context, and the
exchange is a real gloo all-reduce.  What this covers is the sequencing, the schedule and the layout of the exchanged
buffer; the library's own partial-sum and finish kernels are covered on one GPU (test_parity_gpu.py drives the same
loop over two real contexts).  The result must equal a single-process oracle run over all K workers: same rounds, same
parameters (up to the summation order of the mean)."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import qsr_oracle as O
from paper_2310_14423_b200 import binding as B
from paper_2310_14423_b200 import build as qsr_build
from paper_2310_14423_b200 import sharded
from paper_2310_14423_b200 import workloads as W


class OracleEngine:
    """The methods `run_rounds` needs, over the oracle's rows k0 .. k0+rows-1.  The partial sums use the library's
    layout: the parameter sums first, then (state mode AVERAGE) those of state1 and state2, each region starting at a
    multiple of P rounded up to 4 floats."""

    def __init__(self, w, lam, ths, rows, k0):
        self.w = w
        self.cfg = B.make_config(w, K=rows, worker_offset=k0)
        self.S = O.State(w, lam, ths, rows=rows, k0=k0)
        self.P4 = (w.P + 3) // 4 * 4
        self.arrays = [self.S.theta]
        if w.state_sync == W.STATE_AVERAGE:
            self.arrays += [self.S.s1] + ([self.S.s2] if w.opt == W.OPT_ADAMW else [])

    def qsr_sync_sum_floats(self):
        return len(self.arrays) * self.P4

    def qsr_round_length(self, t):
        return B.qsr_config_round_length(self.cfg, t)

    def qsr_local_step(self, t):
        self.S.local_step(t)

    def qsr_local_step_partial(self, t, sums):
        self.S.local_step(t)
        sums.zero_()
        for a, x in enumerate(self.arrays):
            sums[a * self.P4:a * self.P4 + self.w.P] = torch.from_numpy(x.sum(axis=0))

    def qsr_sync_finish(self, sums, K_total, t_next):
        for a, x in enumerate(self.arrays):
            x[:] = sums[a * self.P4:a * self.P4 + self.w.P].numpy() / K_total
        if self.w.state_sync == W.STATE_RESET:
            self.S.s1[:] = 0
            self.S.s2[:] = 0
            self.S.t_state_origin = t_next


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, opt, mode, K_total, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = W.tiny_workload(opt, K=K_total, P=301, T=40, state_sync=mode)
        lam, ths = W.draw_inputs(w.P, w.data_seed)
        rows, k0 = sharded.shard(K_total, world, rank)
        eng = OracleEngine(w, lam, ths, rows, k0)
        sums = torch.zeros(eng.qsr_sync_sum_floats(), dtype=torch.float64)
        rounds = sharded.run_rounds(eng, sums, K_total, 0, w.T, lambda buf: dist.all_reduce(buf))
        np.save(os.path.join(out_dir, f"theta_{rank}.npy"), eng.S.theta)
        np.save(os.path.join(out_dir, f"s1_{rank}.npy"), eng.S.s1)
        np.save(os.path.join(out_dir, f"s2_{rank}.npy"), eng.S.s2)
        np.save(os.path.join(out_dir, f"rounds_{rank}.npy"), np.asarray(rounds, np.int64))
    finally:
        dist.destroy_process_group()


@pytest.fixture(scope="module", autouse=True)
def _built():
    qsr_build.build()


def test_shard_blocks_cover_all_workers():
    for K, world in ((16, 2), (16, 8), (7, 3), (5, 5), (128, 8)):
        blocks = [sharded.shard(K, world, r) for r in range(world)]
        assert sum(b[0] for b in blocks) == K
        assert blocks[0][1] == 0
        for (n0, o0), (n1, o1) in zip(blocks, blocks[1:]):
            assert o1 == o0 + n0 and abs(n0 - n1) <= 1
    with pytest.raises(ValueError):
        sharded.shard(2, 3, 0)


@pytest.mark.parametrize("world,K_total,opt,mode", [
    (2, 6, W.OPT_ADAMW, W.STATE_KEEP),
    (2, 4, W.OPT_SGDM, W.STATE_KEEP),
    (3, 7, W.OPT_ADAMW, W.STATE_RESET),
    (2, 6, W.OPT_ADAMW, W.STATE_AVERAGE),        # three regions in the exchanged buffer
    (3, 7, W.OPT_ADAMW, W.STATE_AVERAGE),        # uneven shards: 3 + 2 + 2 workers
    (3, 7, W.OPT_SGDM, W.STATE_AVERAGE),         # two regions
])
def test_sharded_rounds_equal_single_process(tmp_path, world, K_total, opt, mode):
    port = _free_port()
    mp.spawn(_rank_main, args=(world, port, opt, mode, K_total, str(tmp_path)), nprocs=world, join=True)
    w = W.tiny_workload(opt, K=K_total, P=301, T=40, state_sync=mode)
    lam, ths = W.draw_inputs(w.P, w.data_seed)
    ref = O.State(w, lam, ths)
    st, H = ref.run()
    for r in range(world):
        rounds = np.load(tmp_path / f"rounds_{r}.npy")
        assert np.array_equal(rounds[:, 0], st) and np.array_equal(rounds[:, 1], H)
        theta = np.load(tmp_path / f"theta_{r}.npy")
        rows, k0 = sharded.shard(K_total, world, r)
        assert theta.shape[0] == rows
        np.testing.assert_allclose(theta, ref.theta[k0:k0 + rows], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(np.load(tmp_path / f"s1_{r}.npy"), ref.s1[k0:k0 + rows], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(np.load(tmp_path / f"s2_{r}.npy"), ref.s2[k0:k0 + rows], rtol=1e-12, atol=1e-14)

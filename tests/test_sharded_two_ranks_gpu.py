"""Two processes, one rank each, sharing cuda:0: the replica-sharded path with the library's own kernels in every rank.

Each rank holds a block of the workers in its own CUDA context and runs the product's round loop
(`sharded.run_steps`); the exchange at a round end is a real `torch.distributed` all-reduce of the device buffer the
partial-sum launch wrote (gloo, which stages device tensors through the host; NCCL needs one GPU per rank).  No kernel
waits on another rank: the ranks meet only in the collective, on the host.  Checked: every rank's rows against a
single-process oracle run over all workers, in every state mode, with uneven shards; and `bench.py`'s whole N = 2
flow (rank layout, timed loop, max over ranks, end-to-end leg, only rank 0 reporting) with real launches.
"""
import argparse
import json
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from paper_2310_14423_b200 import binding as B          # noqa: E402
from paper_2310_14423_b200 import sharded               # noqa: E402
from paper_2310_14423_b200 import workloads as W        # noqa: E402

pytestmark = pytest.mark.gpu


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _workload(opt, mode, K_total):
    return W.tiny_workload(opt, K=K_total, P=30001, T=40, state_sync=mode)


def _shard_main(rank, world, port, opt, mode, K_total, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    torch.cuda.set_device(0)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        w = _workload(opt, mode, K_total)
        lam, ths = W.draw_inputs(w.P, w.data_seed)
        rows, k0 = sharded.shard(K_total, world, rank)
        P4 = (w.P + 3) // 4 * 4
        dev = torch.device("cuda", 0)
        theta = torch.zeros(rows, P4, device=dev)
        s1 = torch.zeros(rows, P4, device=dev)
        s2 = torch.zeros(rows, P4, device=dev) if opt == W.OPT_ADAMW else None
        lam_d = torch.zeros(P4, device=dev)
        ths_d = torch.zeros(P4, device=dev)
        lam_d[:w.P] = torch.from_numpy(lam).to(dev)
        ths_d[:w.P] = torch.from_numpy(ths).to(dev)
        ctx = B.Context(B.make_config(w, K=rows, worker_offset=k0, row_stride=P4), theta, s1, s2, lam_d, ths_d,
                        stream=torch.cuda.current_stream().cuda_stream)
        sums = torch.zeros(ctx.qsr_sync_sum_floats(), device=dev)
        rounds = sharded.run_steps(ctx, 0, w.T, sharded.Exchange(sums, K_total, lambda buf: dist.all_reduce(buf)),
                                   whole_rounds=True)
        torch.cuda.synchronize()
        ctx.close()
        np.save(os.path.join(out_dir, f"theta_{rank}.npy"), theta[:, :w.P].cpu().numpy())
        np.save(os.path.join(out_dir, f"s1_{rank}.npy"), s1[:, :w.P].cpu().numpy())
        np.save(os.path.join(out_dir, f"rounds_{rank}.npy"), np.asarray(rounds, np.int64))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("world,K_total,opt,mode", [
    (2, 6, W.OPT_ADAMW, W.STATE_KEEP),
    (2, 5, W.OPT_SGDM, W.STATE_KEEP),            # 3 + 2 workers
    (2, 5, W.OPT_ADAMW, W.STATE_AVERAGE),        # three regions in the exchanged buffer
    (2, 4, W.OPT_ADAMW, W.STATE_RESET),
])
def test_two_ranks_with_real_contexts_equal_the_oracle(tmp_path, world, K_total, opt, mode):
    import gpu_harness as G
    from oracle import qsr_oracle as O
    assert torch.cuda.is_available()
    mp.spawn(_shard_main, args=(world, _free_port(), opt, mode, K_total, str(tmp_path)), nprocs=world, join=True)
    w = _workload(opt, mode, K_total)
    lam, ths = W.draw_inputs(w.P, w.data_seed)
    ref = O.State(w, lam, ths)
    st, H = ref.run()
    for r in range(world):
        rounds = np.load(tmp_path / f"rounds_{r}.npy")
        assert np.array_equal(rounds[:, 0], st) and np.array_equal(rounds[:, 1], H)
        rows, k0 = sharded.shard(K_total, world, r)
        theta = np.load(tmp_path / f"theta_{r}.npy")
        assert theta.shape[0] == rows and (theta == theta[0]).all()
        assert G.rel_err(theta, ref.theta[k0:k0 + rows]) <= G.REL_TOL
        s1 = np.load(tmp_path / f"s1_{r}.npy")
        if mode == W.STATE_RESET:
            assert not s1.any()
        elif mode == W.STATE_AVERAGE:
            assert (s1 == s1[0]).all() and G.rel_err(s1, ref.s1[k0:k0 + rows]) <= 1e-4
        else:
            assert G.rel_err(s1, ref.s1[k0:k0 + rows]) <= 1e-4
    # both ranks end on the same parameters: the exchange gave every rank the global mean
    assert np.array_equal(np.load(tmp_path / "theta_0.npy")[0], np.load(tmp_path / "theta_1.npy")[0])


def _bench_main(rank, world, port, out_dir):
    import bench

    class TwoRanksOneGpu(bench.CudaBackend):
        """bench.py's device backend with both ranks on cuda:0 and gloo in place of NCCL."""

        def __init__(self):
            super().__init__(rank, 0, world)

        def init_process_group(self):
            os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
            dist.init_process_group("gloo", rank=rank, world_size=world)

    args = argparse.Namespace(gpus=world, steps=300, warmup=3, impl="ours", workload="c2", no_cpu_baseline=True,
                              no_e2e=False, packed_rows=False, sharded_path=False, resident_steps=0)
    try:
        out = bench.run_ours(args, TwoRanksOneGpu())
    finally:
        if dist.is_initialized():
            dist.destroy_process_group()
    with open(os.path.join(out_dir, f"bench_{rank}.json"), "w") as f:
        json.dump(out, f)


def test_bench_flow_with_two_ranks_and_real_launches(tmp_path):
    world = 2
    mp.spawn(_bench_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    out = [json.load(open(tmp_path / f"bench_{r}.json")) for r in range(world)]
    assert out[1] is None                                      # only rank 0 reports
    d = out[0]
    base = W.workload("c2")
    assert d["n_gpus"] == 2 and d["config"]["K_total"] == 2 * base.K and d["config"]["K_per_gpu"] == base.K
    assert d["config"]["parallelism"] == "replica-sharded dp2" and d["scaling"] == "weak"
    # c2's first round has 306 steps: steps [0, 300) are plain, so one launch per step on this rank
    assert d["gpu_launches"] == 300 and d["config"]["syncs_in_window"] == 0
    assert d["value"] == pytest.approx(2 * base.K * base.P * 300 / (d["ms_per_step"] * 300 * 1e-3))
    assert d["ms_per_step"] > 0 and d["kernels"]["local_step"]["launches"] == 300
    # the end-to-end leg runs whole rounds through the exchange: it ends on the first round end (306)
    assert d["e2e"]["api"] == "sharded.run_steps" and d["e2e"]["steps"] == 306 and d["e2e"]["value"] > 0

"""World-size-2 checks of the host logic the multi-GPU bench relies on, on CPU with the gloo backend.

The path does not shard across GPUs by communication: every rank runs its own chains on its own GPU with its
own shuffle seeds and the only collective is the MAX over ranks of the timed region.  What can go wrong on the
host is therefore: ranks drawing the same seeds, ranks disagreeing on the workload, and the reduction of the
timings.  The oracle stands in for the GPU here.
"""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import bench
    import oracle
    from paper_2312_08728_b200 import inputs
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        assert bench.dist_env() == (rank, world, rank)
        w = inputs.WORKLOADS["cfg1"].scaled(N=1_000, K=2, epochs=1, T=2)
        host = [inputs.make_buffer(w, k) for k in range(w.K)]
        # every rank sees the same data ...
        digest = torch.tensor([float(host[0][0].double().sum()), float(host[1][1].double().sum())], dtype=torch.float64)
        both = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(both, digest)
        assert all(torch.equal(b, both[0]) for b in both)
        # ... but runs its own chains: the seed rule of the bench
        seed0 = w.seed + rank * 1_000_003
        th = np.zeros(w.p)
        for k, (x, y) in enumerate(host):
            oracle.run_rounds(oracle.LINEAR, x, y, th, w.T, w.n, w.lr, inputs.buffer_seed(seed0, 0, k, w.K))
        mine = torch.from_numpy(th.copy())
        thetas = [torch.zeros_like(mine) for _ in range(world)]
        dist.all_gather(thetas, mine)
        assert not torch.equal(thetas[0], thetas[1])            # different partitions
        assert torch.allclose(thetas[0], thetas[1], atol=0.5)   # same regression problem
        # the timed region is reduced with MAX over ranks
        t = torch.tensor([10.0 + rank, 3.0 - rank], dtype=torch.float64)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        assert t.tolist() == [10.0 + world - 1, 3.0]
        dist.barrier()
        open(os.path.join(out_dir, f"ok{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    procs = [ctx.Process(target=_rank_main, args=(r, world, port, str(tmp_path))) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(300)
    assert all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))


def test_reference_arm_is_rank0_only(tmp_path):
    """Under torchrun only rank 0 runs and prints the reference arm; the others return without work."""
    import subprocess
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, env=env, timeout=300)
    assert p.returncode == 0 and p.stdout.strip() == ""


def test_reference_arm_prints_the_contract_line():
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                        "--steps", "3", "--warmup", "1"], capture_output=True, text=True, env=env, timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    line = json.loads(p.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "sample-grads/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["config"]["workload"].startswith("cfg1")


def test_gpus_flag_starts_the_ranks_itself_and_rank0_alone_prints():
    """`bench.py --gpus 2` with no WORLD_SIZE in the environment starts two ranks on this node; the reference arm
    (the oracle standing in for the GPU) shows it on CPU: exactly one line comes out, from rank 0, with n_gpus = 2."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "cfg1", "--steps", "2", "--warmup", "0"], capture_output=True, text=True, env=env,
                       timeout=600)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, p.stdout
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["impl"] == "reference" and line["value"] > 0
    assert line["cpu_baseline"]["cores"] >= 1


def _split_main(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    import oracle
    from paper_2312_08728_b200 import inputs, multi_gpu
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        Rc = 5  # not a multiple of the world size: shares of 3 and 2 chains
        w = inputs.WORKLOADS["cfg1"].scaled(N=1_200, K=2, epochs=1, T=2, Rc=Rc)
        host = [inputs.make_buffer(w, k) for k in range(w.K)]

        def chain_theta(c):  # the oracle stands in for a GPU working on chain id c
            th = np.zeros(w.p)
            for k, (x, y) in enumerate(host):
                oracle.run_rounds(oracle.LINEAR, x, y, th, w.T, w.n, w.lr, inputs.buffer_seed(w.seed, 0, k, w.K), chain=c)
            return th

        first, count = multi_gpu.chain_share(Rc, world, rank)
        local = torch.from_numpy(np.stack([chain_theta(first + i) for i in range(count)]))
        full = multi_gpu.gather_theta(local, Rc)
        assert tuple(full.shape) == (Rc, w.p)
        if rank == 0:  # N ranks x their shares reproduce the one-process job bit for bit, in chain order
            want = np.stack([chain_theta(c) for c in range(Rc)])
            assert np.array_equal(full.numpy(), want)
        with pytest.raises(ValueError):
            multi_gpu.gather_theta(local[:-1], Rc)  # a share of the wrong length is refused before the collective
        dist.barrier()
        open(os.path.join(out_dir, f"split{rank}"), "w").write("ok")
    finally:
        dist.destroy_process_group()


def test_chains_split_over_two_ranks_and_gathered(tmp_path):
    world = 2
    port = _free_port()
    ctx = mp.get_context("spawn")
    procs = [ctx.Process(target=_split_main, args=(r, world, port, str(tmp_path))) for r in range(world)]
    for p in procs:
        p.start()
    for p in procs:
        p.join(300)
    assert all(p.exitcode == 0 for p in procs), [p.exitcode for p in procs]
    assert all((tmp_path / f"split{r}").exists() for r in range(world))


def test_chain_shares_cover_the_job_exactly():
    from paper_2312_08728_b200.multi_gpu import chain_share
    for Rc in (0, 1, 5, 64, 100):
        for world in (1, 2, 3, 8):
            shares = [chain_share(Rc, world, r) for r in range(world)]
            assert shares[0][0] == 0 and sum(c for _, c in shares) == Rc
            assert all(shares[r][0] + shares[r][1] == shares[r + 1][0] for r in range(world - 1))
            assert max(c for _, c in shares) - min(c for _, c in shares) <= 1
    with pytest.raises(ValueError):
        chain_share(4, 2, 2)

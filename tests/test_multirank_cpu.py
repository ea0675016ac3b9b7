"""The N > 1 path on CPU: two `gloo` ranks.  The path shards by replica (each rank quantizes its
own layer, no data-path collective), so what the ranks share is the timing reduction and the
whole-job value; the reference arm runs on rank 0 only."""
import os
import socket
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from paper_2309_15531_b200 import inputs as I
    dist.init_process_group("gloo", rank=rank, world_size=world)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
    value = bench.whole_job_value(world, 4096 * 4096, ms)
    # every replica builds the same seeded layer: nothing has to be broadcast
    wspec, xspec = I.workload_small()["layers"]["linear"]
    w = I.make_weight(wspec, "cpu").float()
    digest = torch.tensor([float(w.double().sum()), float(w.double().abs().max())], dtype=torch.float64)
    gathered = [torch.zeros_like(digest) for _ in range(world)]
    dist.all_gather(gathered, digest)
    same = all(torch.equal(g, gathered[0]) for g in gathered)
    out_q.put((rank, ms, value, same))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_agree_on_time_and_value():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, value, same in got:
        assert ms == 15.0                              # max over ranks, on both
        assert value == 2 * 4096 * 4096 / 15.0e-3      # both replicas' weights over the slowest rank's time
        assert same


def test_single_rank_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(3.5, 1, torch.device("cpu")) == 3.5
    assert bench.whole_job_value(1, 1000, 2.0) == 500000.0


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_launch_count_matches_the_host_logic():
    import bench
    # 64-column panels: one launch for diagonal block 0 (the later blocks are factored inside the update
    # kernels), panel solve while rows remain below, in-group update while panels remain in the group,
    # one rank-256 update in two launches per finished group with columns to its right; the inverse:
    # 16 seeds, 2 x 16 launches at level 64, 2 per pair above (3 above half-size 256: the second step
    # comes in two halves)
    assert bench.launches_per_step(4096, 128) > 0
    n = bench.launches_per_step(4096, 4096)
    assert n == 366                                    # Hessian 2, RTN 1, scorer 3 + 3, factor 261, GPTQ 96

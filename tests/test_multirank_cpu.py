"""The N > 1 path of bench.py on CPU: two gloo ranks (independent replicas: no data-path collective), the
max-over-ranks step time and whole-job value, and the reference arm's rule that only rank 0 works."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    local_ms = 100.0 + 25.0 * rank                       # rank 1 is the slow replica
    ms = bench.max_over_ranks(local_ms, device="cpu")
    value = bench.whole_job_value(1000, world, ms)
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"ms": ms, "value": value, "seed": bench.replica_seed(5, rank)}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_report_the_slowest_replica_and_the_whole_job(tmp_path):
    port = 29500 + os.getpid() % 2000
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    r = [json.load(open(tmp_path / f"r{i}.json")) for i in range(2)]
    assert r[0]["ms"] == r[1]["ms"] == 125.0              # max over ranks, seen by every rank
    assert abs(r[0]["value"] - 2 * 1000 / 0.125) < 1e-9   # units of both replicas / slowest time
    assert r[0]["seed"] != r[1]["seed"]                   # replicas draw different inputs


def test_single_process_needs_no_process_group():
    import bench
    assert bench.max_over_ranks(12.5, device="cpu") == 12.5
    assert bench.whole_job_value(1000, 1, 500.0) == 2000.0


def test_reference_arm_runs_on_rank_0_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""


def test_plain_command_with_gpus_n_spawns_one_replica_per_gpu(tmp_path, capfd):
    """`python bench.py --gpus N` without a launcher starts N replicas itself: each gets its rank, local rank, the
    world size and one rendezvous address; rank 0's output is the job's output."""
    import bench
    code = ("import os, sys; r = os.environ['RANK']; "
            "open(os.path.join(sys.argv[1], 'rank' + r), 'w').write(' '.join(os.environ[k] for k in "
            "('RANK', 'LOCAL_RANK', 'WORLD_SIZE', 'MASTER_ADDR', 'MASTER_PORT'))); print('line from rank', r)")
    rc = bench.spawn_replicas(3, [sys.executable, "-c", code, str(tmp_path)], timeout=60)
    assert rc == 0
    seen = [open(tmp_path / f"rank{r}").read().split() for r in range(3)]
    assert [s[0] for s in seen] == ["0", "1", "2"] and [s[1] for s in seen] == ["0", "1", "2"]
    assert all(s[2] == "3" and s[3] == "127.0.0.1" for s in seen) and len({s[4] for s in seen}) == 1
    assert capfd.readouterr().out.strip() == "line from rank 0"
    assert bench.spawn_replicas(2, [sys.executable, "-c", "import os, sys; sys.exit(int(os.environ['RANK']) * 3)"]) == 3


def test_two_gloo_ranks_through_the_spawn_path(tmp_path):
    """The spawned replicas rendezvous with the environment spawn_replicas gives them (gloo on CPU) and agree on the
    slowest replica's time."""
    import bench
    code = ("import os, sys, json; sys.path.insert(0, sys.argv[2]); import torch.distributed as dist; import bench; "
            "dist.init_process_group('gloo'); r = dist.get_rank(); ms = bench.max_over_ranks(10.0 + r, device='cpu'); "
            "json.dump({'ms': ms, 'world': dist.get_world_size()}, open(os.path.join(sys.argv[1], f'g{r}.json'), 'w')); "
            "dist.barrier(); dist.destroy_process_group()")
    assert bench.spawn_replicas(2, [sys.executable, "-c", code, str(tmp_path), ROOT], timeout=120) == 0
    got = [json.load(open(tmp_path / f"g{r}.json")) for r in range(2)]
    assert got[0] == got[1] == {"ms": 11.0, "world": 2}

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


def _shard_worker(rank, world, port, out_dir):
    """One rank of the sharded aggregate on CPU: numpy float32 stands in for the two device halves, the exchange is the
    engine's own (torch.distributed all-reduce, here on gloo)."""
    import types
    import numpy as np
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from paper_2511_03983_b200.engine import ShardedRoundEngine, shard_range
    S, n_full, n_sub, rows, d = 4, 12, 5, 2, 8
    rng = np.random.default_rng(7)                       # every rank draws the same blueprints and slices
    blueprints = [np.sort(rng.choice(n_full, n_sub, replace=False)) for _ in range(S)]
    subs = [rng.standard_normal((n_sub * rows, d)).astype(np.float32) for _ in range(S)]
    W_full = rng.standard_normal((n_full * rows, d)).astype(np.float32)
    s0, n = shard_range(S, rank, world)
    part = np.zeros_like(W_full)                         # first half: this rank's sums, zeros elsewhere
    for s in range(s0, s0 + n):                          # ascending subnet order, float32 additions
        for j, b in enumerate(blueprints[s]):
            part[b * rows:(b + 1) * rows] += subs[s][j * rows:(j + 1) * rows]
    t = torch.from_numpy(part)
    ShardedRoundEngine._all_reduce(types.SimpleNamespace(world=world), t)       # the exchange
    count = np.zeros(n_full, dtype=np.int64)
    for bp in blueprints:
        count[bp] += 1
    out = W_full.copy()                                  # second half: division by the global coverage
    held = np.repeat(count > 0, rows)
    out[held] = t.numpy()[held] / np.repeat(count, rows)[held].astype(np.float32)[:, None]
    np.save(os.path.join(out_dir, f"shard{rank}.npy"), out)
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_aggregate_over_two_gloo_ranks_equals_the_aggregator(tmp_path):
    """Partial sums per rank, the engine's all-reduce, division by the global counts: both ranks end with the same
    model, which is the aggregator's (Sec. 3.3) result up to the rounding of a differently associated fp32 sum."""
    import numpy as np
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from fp32_mirror import aggregate_f32
    from oracle import twist_oracle as o
    from paper_2511_03983_b200.engine import shard_range
    port = 31500 + os.getpid() % 2000
    mp.spawn(_shard_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    got = [np.load(tmp_path / f"shard{r}.npy") for r in range(2)]
    assert np.array_equal(got[0], got[1])
    S, n_full, n_sub, rows, d = 4, 12, 5, 2, 8
    rng = np.random.default_rng(7)
    blueprints = [np.sort(rng.choice(n_full, n_sub, replace=False)) for _ in range(S)]
    subs = [rng.standard_normal((n_sub * rows, d)).astype(np.float32) for _ in range(S)]
    W_full = rng.standard_normal((n_full * rows, d)).astype(np.float32)
    mirror = aggregate_f32(W_full, subs, blueprints, rows)
    assert np.max(np.abs(got[0] - mirror)) <= 4 * 2.0 ** -24 * np.max(np.abs(mirror)) * S
    want = o.aggregate(W_full.astype(np.float64), [s.astype(np.float64) for s in subs], blueprints, rows)
    assert np.max(np.abs(got[0] - want)) <= 1e-6 * np.max(np.abs(want)) * S
    uncovered = np.setdiff1d(np.arange(n_full), np.concatenate(blueprints))
    for b in uncovered:                                  # rows nobody holds keep their value
        assert np.array_equal(got[0][b * rows:(b + 1) * rows], W_full[b * rows:(b + 1) * rows])
    for world in (1, 2, 4):
        assert [shard_range(8, r, world) for r in range(world)] == [(r * 8 // world, 8 // world) for r in range(world)]
    for bad in ((8, 0, 3), (8, 2, 2), (8, -1, 2)):
        try:
            shard_range(*bad)
            raise AssertionError(bad)
        except ValueError:
            pass

"""The N > 1 host logic (sharding of a tensor list, max/sum over ranks) on CPU with gloo, world size 2."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2604_03298_b200 import runner, synth
    specs = synth.config_specs(2, scale=16)
    mine = runner.shard(specs, rank, world)
    ms = runner.max_over_ranks(10.0 + 5.0 * rank)
    total = runner.sum_over_ranks(sum(s.numel for s in mine))
    out.put((rank, [s.name for s in mine], ms, total))
    dist.barrier()
    dist.destroy_process_group()


def test_shard_and_reduce_world2():
    from paper_2604_03298_b200 import synth
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    specs = synth.config_specs(2, scale=16)
    names = [s.name for s in specs]
    assert sorted(results[0][1] + results[1][1]) == sorted(names)          # disjoint cover
    assert not set(results[0][1]) & set(results[1][1])
    assert results[0][2] == results[1][2] == 15.0                          # max over ranks
    assert results[0][3] == results[1][3] == float(sum(s.numel for s in specs))


def test_single_process_passthrough():
    from paper_2604_03298_b200 import runner
    assert runner.max_over_ranks(3.5) == 3.5
    assert runner.shard(list(range(7)), 1, 3) == [1, 4]


def _bench(*argv):
    import subprocess
    env = dict(os.environ)
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT"):
        env.pop(k, None)
    env["CUDA_VISIBLE_DEVICES"] = ""      # the launcher must count no device here, GPU machine or not
    return subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), *argv], capture_output=True, text=True,
                          timeout=300, env=env)


def test_bench_gpus_n_refuses_to_pretend():
    """`bench.py --gpus N` with fewer than N devices exits non-zero with a message; it never prints a line."""
    r = _bench("--gpus", "2")
    assert r.returncode != 0
    assert "needs 2 CUDA devices" in r.stderr
    assert r.stdout.strip() == ""


def test_bench_gpus_n_starts_n_ranks():
    """The launcher path of `bench.py --gpus 2`: two ranks rendezvous (gloo, no GPU work), rank 0 prints one
    line with n_gpus = the ranks that really ran."""
    import json
    r = _bench("--gpus", "2", "--spawn-selftest")
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    rec = json.loads(lines[0])
    assert rec["n_gpus"] == 2 and rec["max_over_ranks"] == 11.0 and rec["sum_over_ranks"] == 200.0

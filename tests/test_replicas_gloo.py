"""The N > 1 plumbing of bench.py (independent replicas, max-over-ranks timing, rank-0 report)
on two CPU processes over gloo."""
import json
import os
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_two_replicas_reduce_to_the_slowest_rank(tmp_path):
    script = tmp_path / "ranks.py"
    script.write_text(
        "import json, os, sys\n"
        f"sys.path.insert(0, {ROOT!r})\n"
        "import bench\n"
        "from paper_2608_22643_b200 import synth\n"
        "dist = bench.init_replicas('gloo')\n"
        "rank = int(os.environ['RANK'])\n"
        "cfg = bench.replica_config(synth.CONFIGS['tiny'], rank)\n"
        "ms = bench.max_over_ranks(dist, [10.0 + 5.0 * rank, 3.0 - rank], 'cpu')\n"
        "x = synth.hidden_states(cfg, 2)\n"
        "from paper_2608_22643_b200 import binding as nb\n"
        "threads = nb.replica_host_threads(int(os.environ['WORLD_SIZE']))\n"
        "print(json.dumps({'rank': rank, 'seed': cfg.seed, 'ms': ms, 'x0': float(x.float().sum()), 'threads': threads}))\n"
        "bench.finish_replicas(dist)\n")
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29611", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script)], env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for pr in procs:
        o, e = pr.communicate(timeout=120)
        assert pr.returncode == 0, e
        outs.append(json.loads(o.strip().splitlines()[-1]))
    outs.sort(key=lambda d: d["rank"])
    assert outs[0]["ms"] == outs[1]["ms"] == [15.0, 3.0]          # every rank sees the slowest rank's time
    assert outs[0]["seed"] != outs[1]["seed"] and outs[0]["x0"] != outs[1]["x0"]   # own sequence per replica
    # the replicas of one host share its cores: together their packing threads stay within them
    cores = os.cpu_count() or 1
    assert all(o["threads"] >= 1 for o in outs)
    assert sum(o["threads"] for o in outs) <= max(2, cores - 2)


def test_packing_threads_are_divided_among_replicas():
    sys.path.insert(0, ROOT)
    from paper_2608_22643_b200 import binding as nb
    cores = os.cpu_count() or 1
    assert nb.replica_host_threads(1) == max(1, cores - 2)
    for n in (2, 4, 8):
        assert 1 <= nb.replica_host_threads(n) <= max(1, (cores - 2) // n)
        assert n * nb.replica_host_threads(n) <= max(n, cores - 2)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_store_shrinks_when_the_host_refuses_to_pin_it():
    """bench.py's store sizing: a refusal to page-lock the store makes it retry with three quarters of the layers
    (the stack then reads layer l mod Lp), not below an eighth of the stack or the dense prefix; other errors
    and fixed layer counts are passed on."""
    sys.path.insert(0, ROOT)
    import bench
    from paper_2608_22643_b200 import synth
    cfg = synth.CONFIGS["70b"]
    asked = []

    def fake(cfg_, dev, pin, store_layers):
        asked.append(store_layers)
        if store_layers > 50:
            raise RuntimeError("cudaHostRegister failed with 2")
        return "w1", "w2", "store", 0.5

    out = bench.make_pinned_workload(cfg, 74, "host has 195 GiB available", make=fake)
    assert asked == [74, 55, 41] and out[4] == 41 and "refused to page-lock 55 layers" in out[5]
    asked.clear()
    with pytest.raises(RuntimeError):
        bench.make_pinned_workload(cfg, 74, "", may_shrink=False, make=fake)
    assert asked == [74]
    with pytest.raises(RuntimeError):          # never below the dense prefix
        bench.make_pinned_workload(cfg, 74, "", floor_layers=60, make=fake)

    def other(cfg_, dev, pin, store_layers):
        raise RuntimeError("out of memory")
    with pytest.raises(RuntimeError, match="out of memory"):
        bench.make_pinned_workload(cfg, 74, "", make=other)

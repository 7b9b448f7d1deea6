"""The N > 1 path on CPU: two gloo ranks reduce their timings with a max and own disjoint shards."""
import os

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_37852_b200 import replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    times = [10.0 + rank, 5.0 - rank]                      # rank 1 is slower on the first, faster on the second
    red = replicas.max_over_ranks(times)
    b, e = replicas.shard_units(8 * 2, world, rank)        # 2 batches x 8 KV heads
    out[rank] = (red, (b, e))
    dist.barrier()
    dist.destroy_process_group()


def test_two_rank_max_and_shards():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, 29641, out), nprocs=world, join=True)
    assert out[0][0] == [11.0, 5.0] and out[1][0] == [11.0, 5.0]
    (b0, e0), (b1, e1) = out[0][1], out[1][1]
    assert (b0, e0, b1, e1) == (0, 8, 8, 16)
    assert replicas.aggregate_rate(3.0, 2, 1.5) == 4.0


def test_shard_units_cover_everything_once():
    for n in (1, 7, 16, 33):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                b, e = replicas.shard_units(n, world, r)
                seen += list(range(b, e))
            assert seen == list(range(n))
    with pytest.raises(ValueError):
        replicas.shard_units(4, 2, 2)
    assert replicas.max_over_ranks([1.0, 2.0]) == [1.0, 2.0]   # no process group: identity


def test_launch_local_starts_one_process_per_rank(tmp_path):
    """The launcher behind ``bench.py --gpus N``: N processes with RANK / WORLD_SIZE set, rendezvous on
    127.0.0.1; here two gloo ranks on the CPU reduce a timing with a max and write what they saw."""
    import json
    import sys
    script = tmp_path / "rank.py"
    script.write_text(
        "import json, os, sys\n"
        "import torch.distributed as dist\n"
        f"sys.path.insert(0, {os.path.dirname(os.path.dirname(os.path.abspath(__file__)))!r})\n"
        "from paper_2609_37852_b200 import replicas\n"
        "rank, world = int(os.environ['RANK']), int(os.environ['WORLD_SIZE'])\n"
        "dist.init_process_group('gloo')\n"
        "t = replicas.max_over_ranks([1.0 + rank])[0]\n"
        "rate = replicas.aggregate_rate(6.0, world, t)\n"
        "json.dump({'rank': rank, 'world': world, 't': t, 'rate': rate}, open(sys.argv[1] + str(rank), 'w'))\n"
        "dist.barrier(); dist.destroy_process_group()\n")
    rc = replicas.launch_local(2, str(script), [str(tmp_path / "out")])
    assert rc == 0
    seen = [json.load(open(str(tmp_path / "out") + str(r))) for r in range(2)]
    assert [s["rank"] for s in seen] == [0, 1] and all(s["world"] == 2 for s in seen)
    assert all(s["t"] == 2.0 and s["rate"] == 6.0 for s in seen)         # slowest rank: 2 s; 2 x 6 units / 2 s


def test_bench_gpus_flag_starts_the_ranks_itself():
    """``python bench.py --gpus 2`` with no launcher around it: the reference arm (CPU oracle, rank 0 only)
    prints one line that says n_gpus 2."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--steps", "1",
                        "--warmup", "0"], capture_output=True, text=True, env=env, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["impl"] == "reference" and line["value"] > 0

"""The benchmark's multi-GPU path on CPU: two gloo ranks.  The decode path shards over independent replicas, so
what ranks exchange is a barrier and the maximum of their device times; these tests run exactly that code
(paper_2601_21686_b200/replicas.py) in a world of two, and the reference arm of bench.py under a two-rank launch
(rank 0 alone works and prints, the other exits 0 without output)."""
import json
import os
import socket
import subprocess
import sys

import torch
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    sys.path.insert(0, ROOT)
    from paper_2601_21686_b200 import replicas as R
    me = R.replica_from_env()
    assert (me.rank, me.world, me.local_rank) == (rank, world, rank)
    R.init(me, "gloo")
    R.barrier(me)
    # each rank "measured" different times: the job is as slow as its slowest rank, element by element
    mine = [10.0 + rank, 5.0 - rank, 7.0]
    got = R.max_over_ranks(me, mine)
    rate = R.whole_job_rate(me, units_per_rank=100.0, seconds=got[0])
    with open(os.path.join(out_dir, f"r{rank}.json"), "w") as f:
        json.dump({"max": got, "rate": rate, "root": me.is_root}, f)
    R.finish(me)


def test_max_over_ranks_and_whole_job_rate_in_a_world_of_two(tmp_path):
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    res = [json.load(open(tmp_path / f"r{r}.json")) for r in range(2)]
    for r in res:
        assert r["max"] == [11.0, 5.0, 7.0]
        assert abs(r["rate"] - 2 * 100.0 / 11.0) < 1e-12          # whole-job aggregate over both replicas
    assert [r["root"] for r in res] == [True, False]


def test_single_process_is_a_world_of_one():
    sys.path.insert(0, ROOT)
    from paper_2601_21686_b200 import replicas as R
    me = R.Replica(0, 1, 0)
    assert R.max_over_ranks(me, [3.0, 1.0]) == [3.0, 1.0] and R.whole_job_rate(me, 10.0, 2.0) == 5.0
    R.barrier(me)
    R.finish(me)


def test_reference_arm_under_two_ranks_prints_one_line():
    # bench.py --impl reference as the driver launches it for N = 2: rank 0 times the oracle, rank 1 exits 0 silently
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                                       "--steps", "1", "--warmup", "1"], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=600) for p in procs]
    assert [p.returncode for p in procs] == [0, 0], outs
    lines0 = [l for l in outs[0][0].splitlines() if l.strip()]
    assert len(lines0) == 1 and outs[1][0].strip() == ""
    d = json.loads(lines0[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["e2e"]["h2d_bytes_per_step"] == 0
    assert d["metric"] == "decode_attn_effective_hbm_gbs" and d["unit"] == "GB/s"

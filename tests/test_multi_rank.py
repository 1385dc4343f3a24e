"""The N > 1 path of bench.py on CPU: two gloo ranks.  Every rank runs its own replica of the workload
(rank-seeded, no collective on the data path); times are reduced with MAX and the value is the whole job's."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["DQ_ROOT"])
import torch, torch.distributed as dist
import bench, dq_workloads as wl
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
# each rank reports a different local time; the job's time is the slowest rank's
local = [10.0 + 5.0 * rank, 3.0 - rank, 7.0]
red = bench.max_over_ranks(local)
cfg = wl.by_name("tiny", seed=rank)
g0 = cfg.grad(0)
s = torch.tensor([float(g0[:64].sum())], dtype=torch.float64)
gathered = [torch.zeros_like(s) for _ in range(world)]
dist.all_gather(gathered, s)
dist.barrier()
if rank == 0:
    print(json.dumps({"red": red, "sums": [float(x) for x in gathered],
                      "value": bench.whole_job_value(1000, world, red[0])}))
dist.destroy_process_group()
"""


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_reduce_times_and_seed_replicas(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DQ_ROOT=str(ROOT))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=180) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["red"] == [15.0, 3.0, 7.0]                       # MAX over ranks, element-wise
    assert line["sums"][0] != line["sums"][1]                    # replicas are seeded per rank
    assert line["value"] == 2 * 1000 / 15.0 / 1e6                # whole-job aggregate over both ranks
    assert outs[1][0].strip() == ""                              # only rank 0 prints


def test_reference_arm_prints_only_on_rank_zero():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "1"], env=env, capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    out = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                          "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr
    line = json.loads(out.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["value"] > 0


def test_single_process_reduce_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]


RANGE_WORKER = r"""
import os, sys, json
sys.path.insert(0, os.environ["DQ_ROOT"])
import numpy as np
import torch, torch.distributed as dist
import oracle
from paper_1904_01197_b200.binding import bucket_ranges
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
oracle.build()
n, bucket, step, W = 7 * 512 + 300, 512, 5, 3
rng = np.random.default_rng(123)                       # every rank draws the same data and keeps its own range
side = rng.standard_normal(n).astype(np.float32)
grads = [(side + 0.1 * rng.standard_normal(n)).astype(np.float32) for _ in range(W)]
lo, cnt = bucket_ranges(n, bucket, world)[rank]
msgs, words, scales = [], [], []
for w, g in enumerate(grads):
    if w == 0:
        pk, sc = oracle.dqsg_encode(g[lo:lo + cnt], 900 + w, w, step, bucket, 3, 5, i0=lo)
        msgs.append(oracle.Msg(pk, sc, 900 + w, w, 0, bucket, 3, 5, 0, 0.0, 1.0))
    else:
        pk, sc = oracle.ndqsg_encode(g[lo:lo + cnt], 900 + w, w, step, bucket, 2, 4, 2.0, 1.0, i0=lo)
        msgs.append(oracle.Msg(pk, sc, 900 + w, w, 1, bucket, 2, 0, 4, 2.0, 1.0))
    words.append(pk); scales.append(sc)
mean = oracle.decode_aggregate(msgs, cnt, step, side_info=side[lo:lo + cnt], i0=lo)
mine = {"lo": lo, "cnt": cnt, "words": [x.tolist() for x in words], "scales": [x.view(np.uint32).tolist() for x in scales],
        "mean": mean.view(np.uint32).tolist()}
everyone = [None] * world
dist.all_gather_object(everyone, mine)                 # test plumbing only: the data path has no exchange step
if rank == 0:
    ok = True
    whole_msgs = []
    for w, g in enumerate(grads):
        if w == 0:
            pk, sc = oracle.dqsg_encode(g, 900 + w, w, step, bucket, 3, 5)
            whole_msgs.append(oracle.Msg(pk, sc, 900 + w, w, 0, bucket, 3, 5, 0, 0.0, 1.0))
        else:
            pk, sc = oracle.ndqsg_encode(g, 900 + w, w, step, bucket, 2, 4, 2.0, 1.0)
            whole_msgs.append(oracle.Msg(pk, sc, 900 + w, w, 1, bucket, 2, 0, 4, 2.0, 1.0))
        cat_w = np.concatenate([np.array(e["words"][w], dtype=np.uint32) for e in everyone])
        cat_s = np.concatenate([np.array(e["scales"][w], dtype=np.uint32) for e in everyone])
        ok = ok and np.array_equal(cat_w, pk) and np.array_equal(cat_s, sc.view(np.uint32))
    whole = oracle.decode_aggregate(whole_msgs, n, step, side_info=side)
    cat_m = np.concatenate([np.array(e["mean"], dtype=np.uint32) for e in everyone])
    ok = ok and np.array_equal(cat_m, whole.view(np.uint32))
    print(json.dumps({"ok": bool(ok), "ranges": [[e["lo"], e["cnt"]] for e in everyone]}))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_shard_a_gradient_by_bucket_ranges(tmp_path):
    """Each rank takes one bucket range of every message (the partition of bucket_ranges): the pieces concatenate to
    the whole messages and the whole mean, bit for bit, with no exchange on the data path."""
    script = tmp_path / "range_worker.py"
    script.write_text(RANGE_WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), WORLD_SIZE="2", LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), DQ_ROOT=str(ROOT))
        procs.append(subprocess.Popen([sys.executable, str(script)], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    outs = [p.communicate(timeout=240) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["ok"] is True
    assert line["ranges"] == [[0, 4 * 512], [4 * 512, 3 * 512 + 300]]


def test_bucket_ranges_partition():
    sys.path.insert(0, str(ROOT))
    from paper_1904_01197_b200.binding import bucket_ranges
    for n, bucket, parts in [(0, 512, 3), (1, 512, 4), (25_557_032, 2048, 8), (4096, 2048, 5), (10_000, 96, 7)]:
        r = bucket_ranges(n, bucket, parts)
        assert len(r) == parts and r[0][0] == 0 and sum(c for _, c in r) == n
        for (lo, cnt), (lo2, _) in zip(r, r[1:]):
            assert lo + cnt == lo2
        assert all(lo % bucket == 0 for lo, cnt in r if cnt)
        counts = [-(-c // bucket) for _, c in r]
        assert max(counts) - min(counts) <= 1

"""The N > 1 path of bench.py on CPU: two gloo ranks, each with its own shard of sequences,
meet at a barrier, reduce their times with a maximum and rank 0 reports the whole-job rate.
The path has no data exchange (independent sequences), so this is all the multi-rank logic."""
import json
import os
import socket
import subprocess
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
from paper_2412_12639_b200 import dist as fdist, synth

dist.init_process_group("gloo")
info = fdist.rank_info()
assert info.world == dist.get_world_size() == 2 and info.rank == dist.get_rank()
spec = synth.SPECS["tiny"]
tb = synth.make_trees(spec, seed=fdist.shard_seed(spec.seed, info.rank))
dist.barrier()
# each rank reports a different fake duration; the slower one must win on every rank
mine = [10.0 + 5.0 * info.rank, 3.0 - info.rank, 7.0]
slow = fdist.max_over_ranks(mine)
ok_all = fdist.all_ok(True)
ok_one = fdist.all_ok(info.rank != 1)      # rank 1 reports a failure: everyone must see it
out = {"rank": info.rank, "slow": slow, "ok_all": ok_all, "ok_one": ok_one,
       "nodes": int(tb.total_nodes), "token_sum": int(tb.token.astype("int64").sum()), "prefix": tb.prefix_len.tolist(),
       "rate": fdist.whole_job_rate(1.0, info.world, slow[0])}
print("RESULT " + json.dumps(out), flush=True)
dist.barrier()
dist.destroy_process_group()
"""


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_shard_and_reduce(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    port = _free_port()
    procs = []
    for rank in range(2):
        env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port), OMP_NUM_THREADS="1")
        procs.append(subprocess.Popen([sys.executable, str(script), ROOT], env=env, stdout=subprocess.PIPE,
                                      stderr=subprocess.PIPE, text=True))
    results = {}
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err[-2000:]
        line = [ln for ln in out.splitlines() if ln.startswith("RESULT ")][0]
        r = json.loads(line[len("RESULT "):])
        results[r["rank"]] = r
    assert set(results) == {0, 1}
    for r in results.values():
        assert r["slow"] == [15.0, 3.0, 7.0]            # element-wise maximum, identical on both ranks
        assert r["ok_all"] is True and r["ok_one"] is False
        assert r["rate"] == 2 * 1e3 / 15.0               # both ranks' steps over the slower rank's time
    # the two shards are different batches
    a, b = results[0], results[1]
    assert (a["nodes"], a["token_sum"], a["prefix"]) != (b["nodes"], b["token_sum"], b["prefix"])


def test_single_process_passthrough():
    from paper_2412_12639_b200 import dist as fdist
    assert fdist.max_over_ranks([1.5, 2.0]) == [1.5, 2.0]
    assert fdist.all_ok(True) and not fdist.all_ok(False)
    assert fdist.whole_job_rate(1.0, 4, 2.0) == 2000.0
    assert fdist.shard_seed(7, 3) == 10
    np.testing.assert_raises(ValueError, fdist.whole_job_rate, 1.0, 1, 0.0)


def test_reference_arm_other_ranks_do_no_work():
    """Under a multi-rank launch only rank 0 runs the reference arm; the others exit 0 without output."""
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0", "--workload", "tiny"], env=env, capture_output=True,
                       text=True, timeout=300)
    assert p.returncode == 0, p.stderr[-2000:]
    assert p.stdout.strip() == ""

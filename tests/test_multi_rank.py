"""The N > 1 plumbing of bench.py on CPU: two gloo ranks, distinct substreams per rank, max-over-ranks
timing, and the reference arm printing from rank 0 only.  The data path itself never crosses ranks
(replicas only), so there is nothing else to exchange."""
import json
import os
import subprocess
import sys
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import os, sys, json
sys.path.insert(0, %r)
import numpy as np
import torch.distributed as dist
import bench
from paper_2211_10280_b200 import synth
rank = int(os.environ["RANK"])
dist.init_process_group("gloo")
wl = synth.scaled(synth.TINY, batches=4)
toks, counts = bench.rank_streams(wl, rank, 3)
ms = bench.max_over_ranks(10.0 + 5.0 * rank, dist, "cpu")
dist.barrier()
out = {"rank": rank, "ms": ms, "tok_sum": int(toks.sum()), "shape": list(toks.shape), "counts": int(counts.sum())}
open(sys.argv[1] + f".{rank}", "w").write(json.dumps(out))
dist.destroy_process_group()
"""


def test_two_gloo_ranks_use_distinct_streams_and_report_the_slowest(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % str(ROOT))
    out = tmp_path / "out"
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    subprocess.check_call([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                           "--master-addr", "127.0.0.1", "--master-port", "29611", str(script), str(out)],
                          env=env, cwd=str(ROOT), timeout=300)
    r = [json.loads(Path(f"{out}.{i}").read_text()) for i in range(2)]
    assert r[0]["ms"] == r[1]["ms"] == 15.0
    assert r[0]["shape"] == r[1]["shape"] == [3, 1, 512]
    assert r[0]["tok_sum"] != r[1]["tok_sum"]
    assert r[0]["counts"] == r[1]["counts"] == 10_000 + 4 * 512


def test_reference_arm_prints_one_line_from_rank_zero(tmp_path):
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "sgns_tiny",
                          "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True, timeout=300)
    assert res.returncode == 0 and res.stdout.strip() == ""
    env = dict(os.environ, RANK="0", WORLD_SIZE="2", LOCAL_RANK="0")
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--workload", "sgns_tiny",
                          "--steps", "2", "--warmup", "1", "--gpus", "2"], env=env, capture_output=True, text=True,
                         timeout=300)
    assert res.returncode == 0
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "pairs/s" and line["value"] > 0
    assert line["config"]["workload"] == "sgns_tiny[W=2]" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0


def test_gpus_flag_starts_the_ranks_itself(tmp_path):
    """`bench.py --gpus 2` with no launcher around it (no RANK in the environment) must start two ranks; with the
    reference arm rank 0 alone works and prints the one line, which says n_gpus 2 and names the workload as two
    ranks run it."""
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    res = subprocess.run([sys.executable, str(ROOT / "bench.py"), "--gpus", "2", "--impl", "reference", "--workload",
                          "sgns_tiny", "--steps", "2", "--warmup", "1"], env=env, capture_output=True, text=True,
                         timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(x) for x in res.stdout.splitlines() if x.startswith("{")]
    assert len(lines) == 1
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["value"] > 0
    # sgns_tiny has one replica: over two ranks it runs with one replica per rank
    assert line["config"]["replicas"] == 2 and line["config"]["workload"] == "sgns_tiny[W=2]"


def test_both_arms_print_the_same_config_keys():
    import bench
    from paper_2211_10280_b200 import synth

    a = bench.config_of(synth.LARGE_DASGD, 1, "x")
    assert {"workload", "V", "d", "window", "k", "batch", "replicas", "max_delay", "reduction", "pairs_per_batch",
            "storage", "l2", "parallelism"} <= set(a)
    wl8, local, scaling = bench.sharded_workload(synth.LARGE_DASGD, 8)
    assert (wl8.W, local, scaling) == (8, 1, "weak") and wl8.stream_seeds == tuple(range(2, 10))
    wl2, local, scaling = bench.sharded_workload(synth.LARGE_DASGD, 2)
    assert (wl2.W, local, scaling) == (4, 2, "strong") and wl2 is synth.LARGE_DASGD
    assert bench.repeats_for(110.0) == 19 and bench.repeats_for(5000.0) == 1 and bench.repeats_for(1.0) == bench.MAX_REPEATS

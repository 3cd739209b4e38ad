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
    assert line["config"]["workload"] == "sgns_tiny" and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0

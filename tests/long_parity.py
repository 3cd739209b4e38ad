#!/usr/bin/env python
"""Long parity runs: the CUDA path and the CPU oracle side by side over many steps of a named workload.

    python tests/long_parity.py --workload sgns_mid --steps 2000 [--check-every 100] [--out FILE]

Not collected by pytest (a full-size run takes minutes to half an hour of oracle time); the short run in
test_gpu_parity.py keeps this file exercised.  Every step: every replica trains its batch on both sides (the
sampler is rebuilt on both at the drift boundaries of a drifting workload), the message row ids must be equal, and
both sides must apply the same number of messages.  Every `check_every` steps and after the last: the sampled
negatives of the last batch bit for bit, every replica's delivery log bit for bit, and both tables of every
replica within `tol` (the 200-batch bar of 1e-3 by default) under the measure of parity_utils.rel_err.  Prints one
JSON line: the steps run (T'), the errors at every check, the largest, and the time each side took.
"""
from __future__ import annotations

import argparse
import json
import sys
import time
from pathlib import Path

import numpy as np

ROOT = Path(__file__).resolve().parent.parent
for p in (str(ROOT), str(ROOT / "tests")):
    if p not in sys.path:
        sys.path.insert(0, p)

from parity_utils import make_pair, rel_err  # noqa: E402
from paper_2211_10280_b200 import synth  # noqa: E402


def run(wl: synth.Workload, steps: int, check_every: int, tol: float = 1e-3, replicas_checked=None, log=None) -> dict:
    import torch

    streams = synth.all_streams(wl, steps)
    counts = None if wl.drift_every else synth.stream_counts(synth.all_streams(wl), wl.V)
    o, g = make_pair(wl, counts=counts)
    dstreams = [torch.from_numpy(np.ascontiguousarray(s, dtype=np.int32)).cuda() for s in streams]
    torch.cuda.synchronize()
    checked = list(range(wl.W)) if replicas_checked is None else list(replicas_checked)
    checks, t_oracle, t_gpu, loss_first, loss_last = [], 0.0, 0.0, None, None
    rebuilds = 0
    for t in range(steps):
        if wl.drift_every and t and t % wl.drift_every == 0:
            o.update_sampler()
            g.tensair_update_sampler()
            assert all(np.array_equal(a, b) for a, b in zip(o.sampler(), g.tensair_read_sampler())), \
                f"step {t}: rebuilt sampler tables differ"
            rebuilds += 1
        last = t == steps - 1 or (t + 1) % check_every == 0
        for i in range(wl.W):
            t0 = time.time()
            rc, loss_o, rows_o = o.train_batch(i, streams[i][t], t)
            t_oracle += time.time() - t0
            assert rc == 0
            t0 = time.time()
            loss_g, info = g.tensair_train_batch(i, dstreams[i][t], t, want_loss=True, want_info=True)
            t_gpu += time.time() - t0
            assert info.n_rows == rows_o, f"step {t} replica {i}: {info.n_rows} message rows, oracle {rows_o}"
            assert np.array_equal(o.read_message_ids(i, t), g.tensair_read_message_ids(i, t)), \
                f"step {t} replica {i}: message row ids differ"
            if last:
                assert np.array_equal(o.read_negatives(), g.tensair_read_negatives()), f"step {t}: negatives differ"
            if i == 0:
                loss_first = loss_o if loss_first is None else loss_first
                loss_last = (loss_o, loss_g)
        for j in range(wl.W):
            t0 = time.time()
            n_o = o.apply_messages(j, t)
            t_oracle += time.time() - t0
            assert n_o == g.tensair_apply_messages(j, t), f"step {t} receiver {j}: applied counts differ"
        if last:
            errs = []
            for j in checked:
                assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j)), f"step {t}: delivery log of {j}"
                for which in (0, 1):
                    errs.append(rel_err(g.tensair_read_embeddings(j, which), o.read_embeddings(j, which)))
            checks.append({"step": t + 1, "max_rel_err": max(errs)})
            if log:
                log(f"step {t + 1}: max rel err {max(errs):.3e}, oracle {t_oracle:.0f} s")
            assert max(errs) <= tol, (t + 1, max(errs), tol)
    assert o.drain() == g.tensair_drain()
    errs = []
    for j in checked:
        assert np.array_equal(o.delivery_log(j), g.tensair_read_delivery_log(j)), f"after the drain: delivery log of {j}"
        for which in (0, 1):
            errs.append(rel_err(g.tensair_read_embeddings(j, which), o.read_embeddings(j, which)))
    assert max(errs) <= tol, ("after the drain", max(errs), tol)
    out = {"workload": wl.name, "steps": steps, "replicas": wl.W, "replicas_compared": checked, "tolerance": tol, "checks": checks,
           "max_rel_err": max(c["max_rel_err"] for c in checks), "after_drain": max(errs),
           "sampler_rebuilds": rebuilds, "loss_of_replica_0": {"first": loss_first, "last_oracle": loss_last[0], "last_cuda": loss_last[1]},
           "oracle_seconds": round(t_oracle, 1), "cuda_seconds_with_readbacks": round(t_gpu, 1),
           "delivery_logs": "bit-identical", "message_row_ids": "bit-identical at every step"}
    o.close()
    g.close()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", required=True)
    ap.add_argument("--steps", type=int, required=True)
    ap.add_argument("--check-every", type=int, default=100)
    ap.add_argument("--tol", type=float, default=1e-3)
    ap.add_argument("--out", default="")
    ap.add_argument("--check-replicas", default="", help="comma-separated replicas whose tables and logs are compared (default: all)")
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]
    checked = [int(x) for x in args.check_replicas.split(",")] if args.check_replicas else None
    res = run(wl, args.steps, args.check_every, args.tol, replicas_checked=checked,
              log=lambda m: print(m, file=sys.stderr, flush=True))
    line = json.dumps(res)
    print(line)
    if args.out:
        Path(args.out).write_text(line + "\n")


if __name__ == "__main__":
    main()

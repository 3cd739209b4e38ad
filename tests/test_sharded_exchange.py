"""The message exchange between processes (paper_2211_10280_b200/exchange.py) on CPU: two and three gloo ranks.

No GPU here, so the context is replaced by a stand-in with the same calls: its pool slots are CPU
tensors, its "training" writes a message whose content is a function of (sender, step), and its delivery
schedule is the library's own host-side schedule (tensair_schedule_*).  Checked per rank: every message that
is applied carries the sender's content (it arrived whole, before it was due, and was not overwritten before
use), and every receiver's delivery log - order, due steps and the staleness of Section 3.1 - equals the log
of a one-process schedule over all replicas.
"""
import json
import os
import subprocess
import sys
from pathlib import Path

import numpy as np
import pytest

ROOT = Path(__file__).resolve().parent.parent

WORKER = r"""
import json, os, sys
sys.path.insert(0, %r)
import numpy as np
import torch
import torch.distributed as dist
from paper_2211_10280_b200 import binding as B
from paper_2211_10280_b200.exchange import ShardedReplicas

LOCAL, D, SEED, STEPS, MAX_ROWS, STRIDE = int(sys.argv[2]), 2, 77, 9, 40, 8
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo")
W = world * LOCAL


def content(g, step):
    # what replica g "computes" at `step`: a row count, ascending ids and delta rows, all functions of (g, step)
    rng = np.random.default_rng(1000 * g + step)
    n = int(rng.integers(0, MAX_ROWS + 1))
    ids = np.sort(rng.choice(10_000, size=n, replace=False)).astype(np.int32)
    delta = rng.standard_normal((n, STRIDE)).astype(np.float32)
    return n, int((ids < 5000).sum()), ids, delta


class Port:
    # stands in for binding.Context: same calls, CPU tensors, the library's host-side schedule
    def __init__(self):
        self.sched = B.Schedule(W, D, SEED)
        self.first = rank * LOCAL
        self.slots = {}
        self.held = {}          # slot -> (sender, step, rows) as committed
        self.applied = []       # (receiver, origin, sender, content matches, staleness)

    def _slot(self, g, step):
        key = (g, step %% (D + 1))
        if key not in self.slots:
            self.slots[key] = (torch.full((MAX_ROWS,), -1, dtype=torch.int32), torch.zeros(MAX_ROWS * STRIDE))
        return key

    def train(self, r, step):
        g = self.first + r
        n, n_in, ids, delta = content(g, step)
        key = self._slot(g, step)
        self.slots[key][0][:n] = torch.from_numpy(ids)
        self.slots[key][1][:n * STRIDE] = torch.from_numpy(delta.ravel())
        assert self.sched.on_train(g, step) == B.OK
        self.held[key] = (g, step, n, n_in)

    def tensair_message_rows(self, r, step):
        g, s, n, n_in = self.held[self._slot(self.first + r, step)]
        assert s == step
        return n, n_in

    def tensair_message_buffers(self, g, step):
        return self.slots[self._slot(g, step)]

    def tensair_commit_message(self, g, step, n, n_in, stream=None):
        assert not (self.first <= g < self.first + LOCAL)
        assert self.sched.on_train(g, step) == B.OK, "slot still has recipients"
        self.held[self._slot(g, step)] = (g, step, n, n_in)

    def _check(self, receiver, rec):
        origin, sender = int(rec[0]), int(rec[1])
        n, n_in, ids, delta = content(sender, origin)
        g, s, hn, hin = self.held[self._slot(sender, origin)]
        got_ids, got_delta = self.slots[self._slot(sender, origin)]
        ok = (s == origin and hn == n and hin == n_in and np.array_equal(got_ids[:n].numpy(), ids)
              and np.array_equal(got_delta[:n * STRIDE].numpy(), delta.ravel()))
        self.applied.append((receiver, origin, sender, bool(ok), int(rec[4])))

    def tensair_apply_messages(self, r, step):
        due = self.sched.take_due(self.first + r, step)
        for rec in due:
            self._check(self.first + r, rec)
        return len(due)

    def tensair_apply_step(self, step):
        return sum(self.tensair_apply_messages(r, step) for r in range(LOCAL))

    def tensair_shadow_apply(self, g, step, drain):
        return len(self.sched.take_due(g, step, drain))

    def tensair_drain(self):
        total = 0
        for g in range(W):
            due = self.sched.take_due(g, 0, True)
            if self.first <= g < self.first + LOCAL:
                total += len(due)
                for rec in due:
                    self._check(g, rec)
        return total


port = Port()
OVERLAP = int(sys.argv[3])
grp = ShardedReplicas(port, rank, world, LOCAL, dist=dist, max_delay=D, seed=SEED, overlap=bool(OVERLAP))
logs = {r: [] for r in range(LOCAL)}
for t in range(STEPS):
    for r in range(LOCAL):
        port.train(r, t)
    grp.exchange(t)
    grp.apply(t)
grp.drain()
assert not grp._flying, "a transfer was never waited for"
out = {"rank": rank, "applied": port.applied, "sent": grp.bytes_sent, "received": grp.bytes_received,
       "at_own_step": grp.bytes_waited_at_own_step, "later": grp.bytes_waited_later}
open(sys.argv[1] + f".{rank}", "w").write(json.dumps(out))
dist.barrier()
dist.destroy_process_group()
"""


@pytest.mark.parametrize("world,local,port,overlap", [(2, 1, 29621, 1), (2, 2, 29622, 1), (3, 1, 29623, 1), (2, 1, 29624, 0)])
def test_every_rank_applies_every_message_once_in_the_one_process_order(tmp_path, world, local, port, overlap):
    from paper_2211_10280_b200 import binding as B

    script = tmp_path / "worker.py"
    script.write_text(WORKER % str(ROOT))
    out = tmp_path / "out"
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    subprocess.check_call([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
                           "--master-addr", "127.0.0.1", "--master-port", str(port), str(script), str(out), str(local),
                           str(overlap)],
                          env=env, cwd=str(ROOT), timeout=300)
    res = [json.loads(Path(f"{out}.{r}").read_text()) for r in range(world)]
    W, D, steps = world * local, 2, 9
    # the one-process schedule over all replicas
    ref = B.Schedule(W, D, 77)
    want = {g: [] for g in range(W)}
    for t in range(steps):
        for g in range(W):
            assert ref.on_train(g, t) == B.OK
        for g in range(W):
            want[g] += [(int(r[0]), int(r[1]), int(r[4])) for r in ref.take_due(g, t)]
    for g in range(W):
        want[g] += [(int(r[0]), int(r[1]), int(r[4])) for r in ref.take_due(g, 0, True)]
    for r in range(world):
        got = {g: [] for g in range(r * local, (r + 1) * local)}
        for receiver, origin, sender, ok, staleness in res[r]["applied"]:
            assert ok, f"rank {r}: message ({sender}, {origin}) did not carry the sender's content when applied"
            got[receiver].append((origin, sender, staleness))
        for g in got:
            assert got[g] == want[g], f"replica {g} on rank {r}: order or staleness differs from the one-process schedule"
            assert len(got[g]) == (W - 1) * steps and len(set(got[g])) == len(got[g])
    # every byte sent is received once per other rank
    assert sum(x["sent"] for x in res) == sum(x["received"] for x in res) > 0
    # every received byte was waited for exactly once: at its own step when it was due there, later otherwise
    for x in res:
        assert x["at_own_step"] + x["later"] == x["received"]
        if overlap:
            # delays are uniform in {0, 1, 2}: a good share of what a rank receives is not due at its own step
            assert x["later"] > 0.2 * x["received"]
        else:
            assert x["later"] == 0

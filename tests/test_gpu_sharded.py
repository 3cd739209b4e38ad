"""Replicas spread over several contexts (the placement of Section 2.2: one Model instance per worker, every
gradient sent to every other instance) must compute what one context holding all replicas computes.

One GPU stands in for the workers: each shard is its own context with its own tables and pool, and the
"wire" is a device copy from the sender's pool slot into the slot the receiving context keeps for that
sender - the copy an NCCL broadcast makes between GPUs.  Parity of the one-context job with the oracle is
covered by test_gpu_parity.py, so bit-identity with it carries the oracle's bar over; the message ids and
delivery logs are compared with the oracle directly as well.
"""
import numpy as np
import pytest

from parity_utils import make_pair
from paper_2211_10280_b200 import binding as B
from paper_2211_10280_b200 import synth
from paper_2211_10280_b200.exchange import ShardedReplicas

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch():
    import torch as t

    assert t.cuda.is_available(), "these tests need a CUDA device"
    return t


def dev(torch, a):
    """The batch in device memory, complete when this returns (so that the suite can also run with the knob that lets
    the library start on a batch's tokens ahead of the stream: TENSAIR_TUNE=early_prepare=2)."""
    t = torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    torch.cuda.current_stream().synchronize()
    return t


def shard_contexts(wl, counts, world, local):
    kw = dict(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, W=local, lr=wl.lr, max_delay=wl.max_delay,
              seed=wl.seed, counts=counts, reduction=wl.reduction, world_replicas=world * local)
    return [B.Context(first_replica=p * local, **kw) for p in range(world)]


def wire(shards, local, step):
    """Moves every message of `step` into every other shard's pool and files it there."""
    world = len(shards)
    for g in range(world * local):
        owner, r = divmod(g, local)
        n, n_in = shards[owner].tensair_message_rows(r, step)
        src_ids, src_delta = shards[owner].tensair_message_buffers(g, step)
        stride = src_delta.numel() // src_ids.numel()
        for p in range(world):
            if p == owner:
                continue
            dst_ids, dst_delta = shards[p].tensair_message_buffers(g, step)
            dst_ids[:n].copy_(src_ids[:n])
            dst_delta[:n * stride].copy_(src_delta[:n * stride])
            shards[p].tensair_commit_message(g, step, n, n_in)


@pytest.mark.parametrize("world,local,routed", [(2, 1, False), (2, 2, False), (4, 1, False), (2, 1, True)])
def test_shards_compute_what_one_context_computes(torch, world, local, routed):
    W = world * local
    wl = synth.scaled(synth.LARGE_DASGD, V=30_000, d=300, batch=1024, W=W, stream_seeds=tuple(range(20, 20 + W)),
                      max_delay=2, batches=7)
    streams = synth.all_streams(wl, wl.batches)
    counts = synth.stream_counts(streams, wl.V)
    o, one = make_pair(wl, counts=counts)
    shards = shard_contexts(wl, counts, world, local)
    groups = [ShardedReplicas(shards[p], p, world, local) for p in range(world)]   # apply() and drain() only
    for t in range(wl.batches):
        for g in range(W):
            tok = dev(torch, streams[0 if routed else g][t])
            p, r = divmod(g, local)
            if routed:
                assert o.train_batch_routed(g, streams[0][t], t)[0] == 0
                one.tensair_train_batch_routed(g, tok, t)
                shards[p].tensair_train_batch_routed(r, tok, t)
            else:
                assert o.train_batch(g, streams[g][t], t)[0] == 0
                one.tensair_train_batch(g, tok, t)
                shards[p].tensair_train_batch(r, tok, t)
        wire(shards, local, t)
        for g in range(W):
            p, r = divmod(g, local)
            # every shard holds every message of the step, bit for bit
            ids_one, delta_one = one.tensair_read_message(g, t)
            assert np.array_equal(ids_one, o.read_message(g, t)[0])
            for q in range(world):
                ids_q, delta_q = shards[q].tensair_read_message(g, t)
                assert np.array_equal(ids_q, ids_one)
                assert np.array_equal(delta_q.view(np.uint32), delta_one.view(np.uint32))
        applied_one = sum(one.tensair_apply_messages(j, t) for j in range(W))
        for j in range(W):
            o.apply_messages(j, t)
        assert sum(grp.apply(t) for grp in groups) == applied_one
    assert sum(s.tensair_drain() for s in shards) == one.tensair_drain() == o.drain()
    for g in range(W):
        p, r = divmod(g, local)
        assert shards[p].tensair_pending(r) == 0
        log = shards[p].tensair_read_delivery_log(r)
        assert np.array_equal(log, one.tensair_read_delivery_log(g)), "delivery order or staleness differs"
        assert np.array_equal(log, o.delivery_log(g))
        for which in (0, 1):
            got = shards[p].tensair_read_embeddings(r, which)
            want = one.tensair_read_embeddings(g, which)
            assert np.array_equal(got.view(np.uint32), want.view(np.uint32)), (g, which)
    assert all(s.tensair_sync() == B.OK for s in shards)


def test_a_slot_still_to_be_applied_is_not_handed_out_for_receiving(torch):
    wl = synth.scaled(synth.TINY, V=500, d=8, batch=64, W=1, max_delay=0)
    a, b = shard_contexts(wl, None, 2, 1)
    tok = dev(torch, np.arange(64) % 500)
    a.tensair_train_batch(0, tok, 0)
    n, n_in = a.tensair_message_rows(0, 0)
    ids, delta = b.tensair_message_buffers(0, 0)
    ids[:n].copy_(a.tensair_message_buffers(0, 0)[0][:n])
    b.tensair_commit_message(0, 0, n, n_in)
    with pytest.raises(B.TensairError) as e:          # replica 1 (in b) has not applied (0, 0) yet
        b.tensair_message_buffers(0, 1)
    assert e.value.code == B.EPENDING
    assert b.tensair_apply_messages(0, 0) == 1 and b.tensair_shadow_apply(0, 0) == 0
    b.tensair_message_buffers(0, 1)
    with pytest.raises(B.TensairError) as e:          # a local message that was never built
        a.tensair_message_buffers(0, 5)
    assert e.value.code == B.ENOTFOUND
    with pytest.raises(B.TensairError):               # a local replica's message files itself
        a.tensair_commit_message(0, 1, 0, 0)
    with pytest.raises(B.TensairError):               # a local receiver is applied for real
        a.tensair_shadow_apply(0, 0)


class LoopbackDist:
    """all_gather and broadcast of torch.distributed between THREADS of one process, one thread per shard, all on one
    GPU: a transfer is a device copy enqueued on the receiver's current stream behind an event of the sender's
    stream - what a collective between GPUs does to the streams it is enqueued on.  Every rendezvous has a time
    limit, so a failing thread fails the test instead of stalling it."""

    def __init__(self, torch, world):
        import threading

        self.torch, self.world = torch, world
        self.barrier = threading.Barrier(world, timeout=120)
        self.box = [None] * world
        self.done = [None] * world
        self.me = threading.local()

    def _event(self):
        ev = self.torch.cuda.Event()
        ev.record()                       # on the calling thread's current stream
        return ev

    def _finish(self):
        # nobody reuses a source tensor before every receiver's copy from it has run
        self.done[self.me.rank] = self._event()
        self.barrier.wait()
        for ev in self.done:
            self.torch.cuda.current_stream().wait_event(ev)
        self.barrier.wait()

    def all_gather(self, out, tensor, group=None):
        self.box[self.me.rank] = (tensor, self._event())
        self.barrier.wait()
        for i, (src, ev) in enumerate(self.box):
            self.torch.cuda.current_stream().wait_event(ev)
            out[i].copy_(src)
        self._finish()

    def broadcast(self, tensor, src, group=None, async_op=False):
        if self.me.rank == src:
            self.box[src] = (tensor, self._event())
        self.barrier.wait()
        if self.me.rank != src:
            data, ev = self.box[src]
            self.torch.cuda.current_stream().wait_event(ev)
            tensor.copy_(data)
        self._finish()


@pytest.mark.parametrize("world,local,overlap", [(2, 1, True), (2, 2, True), (4, 1, True), (2, 1, False)])
def test_exchange_on_a_communication_stream_equals_the_one_context_job(torch, world, local, overlap):
    """The exchange layer itself (row counts read on the device, broadcasts and the received messages' indices on a
    communication stream, the training stream waiting only for what is due) driven by one thread per shard over a
    loop-back transport: tables and delivery logs must equal the one-context job bit for bit, and with delays up
    to 2 a good part of what a shard receives must not have been waited for at its own step."""
    import threading

    W = world * local
    wl = synth.scaled(synth.LARGE_DASGD, V=30_000, d=300, batch=1024, W=W, stream_seeds=tuple(range(20, 20 + W)),
                      max_delay=2, batches=9)
    streams = synth.all_streams(wl, wl.batches)
    counts = synth.stream_counts(streams, wl.V)
    kw = dict(V=wl.V, d=wl.d, window=wl.window, k=wl.k, batch=wl.batch, lr=wl.lr, max_delay=wl.max_delay,
              seed=wl.seed, counts=counts, reduction=wl.reduction)
    one = B.Context(W=W, **kw)
    for t in range(wl.batches):
        for g in range(W):
            one.tensair_train_batch(g, dev(torch, streams[g][t]), t)
        one.tensair_apply_step(t)
    one.tensair_drain()

    wire_ = LoopbackDist(torch, world)
    results, errors = [None] * world, []

    def shard(p):
        try:
            wire_.me.rank = p
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                ctx = B.Context(W=local, world_replicas=W, first_replica=p * local, stream=stream, **kw)
                grp = ShardedReplicas(ctx, p, world, local, dist=wire_, count_device="cuda", overlap=overlap)
                toks = [[dev(torch, streams[p * local + r][t]) for r in range(local)] for t in range(wl.batches)]
                for t in range(wl.batches):
                    for r in range(local):
                        ctx.tensair_train_batch(r, toks[t][r], t)
                    grp.exchange(t)
                    grp.apply(t)
                grp.drain()
                assert ctx.tensair_sync() == B.OK and not grp._flying
                results[p] = ([ctx.tensair_read_delivery_log(r) for r in range(local)],
                              [[ctx.tensair_read_embeddings(r, which) for which in (0, 1)] for r in range(local)],
                              (grp.bytes_received, grp.bytes_waited_at_own_step, grp.bytes_waited_later, grp.bytes_sent))
                ctx.close()
        except BaseException as e:          # noqa: BLE001 - reported by the main thread
            errors.append((p, repr(e)))
            wire_.barrier.abort()

    threads = [threading.Thread(target=shard, args=(p,)) for p in range(world)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=600)
    assert not errors, errors
    assert all(r is not None for r in results)
    for p in range(world):
        logs, tables, (received, own_step, later, sent) = results[p]
        for r in range(local):
            g = p * local + r
            assert np.array_equal(logs[r], one.tensair_read_delivery_log(g)), "delivery order or staleness differs"
            for which in (0, 1):
                want = one.tensair_read_embeddings(g, which)
                assert np.array_equal(tables[r][which].view(np.uint32), want.view(np.uint32)), (g, which)
        assert own_step + later == received > 0
        assert (later > 0.2 * received) if overlap else (later == 0)
    assert sum(r[2][3] for r in results) == sum(r[2][0] for r in results)

"""Replicas spread over processes, one GPU each: the message exchange between them.

The paper places one Model instance per worker and has each send its gradient to every other instance
(Section 2.2, data parallelism; Algorithm 1, send_gradients), and a Model goes on computing while gradients
arrive (Section 3.1).  Here a job of `world_size` processes holds `local` replicas each (global id =
rank * local + local index).  Per step every process trains its own replicas, then the messages travel: the
senders' row counts go round in one small all-gather, and each sender's row ids and delta rows are broadcast
straight out of its pool slot into the slot the other processes keep for that sender - no staging copy, no
padding to a common size.  After that every process holds every message in its own GPU memory and applies what
is due with the same kernels as a one-process job; the delivery schedule is a function of the seed, so every
process keeps the whole of it and the result is the one-process result bit for bit.

The transfers run on a communication stream of their own.  The training stream waits for a message only
before the first apply call at which one of this process's replicas needs it: step + the smallest delivery
delay to a local receiver (the delays are a function of the seed, so every process knows them).  A message
that is not due here at its own step therefore travels while the next batch is trained; with delays uniform
in {0, 1, 2} and one replica per process that is two thirds of what a process receives.  Filing a received
message in the delivery schedule (host-side) still happens at once and in the one-process order, so delivery
order and staleness do not depend on when the bytes land.

Only plumbing lives here (torch.distributed calls, streams, events and the order of the library calls); the
arithmetic is the library's.  `port` is a binding.Context created with world_replicas / first_replica, or
anything with the same calls (the CPU tests use a stand-in that needs no GPU; there the "communication
stream" is a list of asynchronous gloo requests).
"""
from __future__ import annotations


class _CudaLane:
    """Transfers on a CUDA stream of their own; a message's completion is an event on that stream."""

    def __init__(self, torch, main_stream):
        self.torch = torch
        self.main = main_stream
        self.stream = torch.cuda.Stream(device=main_stream.device)

    def begin(self):
        """The transfers of a step start after everything the training stream holds so far."""
        ev = self.torch.cuda.Event()
        ev.record(self.main)
        self.stream.wait_event(ev)

    def run(self):
        return self.torch.cuda.stream(self.stream)

    def mark(self, requests):
        ev = self.torch.cuda.Event()
        ev.record(self.stream)
        return ev

    def host_wait(self, requests):
        ev = self.torch.cuda.Event()
        ev.record(self.stream)
        ev.synchronize()

    def stream_wait(self, token):
        self.main.wait_event(token)

    commit_stream = property(lambda self: self.stream)
    async_op = False


class _HostLane:
    """No GPU: transfers are asynchronous requests of the process group; completion = all of them waited for."""

    class _Nothing:
        def __enter__(self):
            return self

        def __exit__(self, *a):
            return False

    def begin(self):
        pass

    def run(self):
        return self._Nothing()

    def mark(self, requests):
        return list(requests)

    def host_wait(self, requests):
        for r in requests:
            r.wait()

    def stream_wait(self, token):
        for r in token:
            r.wait()

    commit_stream = None
    async_op = True


class ShardedReplicas:
    def __init__(self, port, rank: int, world_size: int, local: int, dist=None, group=None, count_device="cpu",
                 max_delay=None, seed=None, delay=None, overlap=True):
        """dist: torch.distributed (initialised); may be None when world_size == 1 or when the caller moves the
        messages itself and uses only apply() and drain().  count_device: where the small tensor of row counts
        lives for the all-gather ("cuda" with nccl, "cpu" with gloo).  max_delay, seed: those of the job's
        configuration (taken from port.cfg when it has one); with them the exchange knows at which step a message
        is first needed here and lets it travel until then.  Without them, or with overlap=False, every message
        is waited for at its own step.  delay: the delay function (step, sender, receiver) -> steps, default the
        library's tensair_delay."""
        self.port, self.rank, self.world_size, self.local = port, rank, world_size, local
        self.dist, self.group, self.count_device = dist, group, count_device
        self.world_replicas = world_size * local
        self.first = rank * local
        cfg = getattr(port, "cfg", None)
        self.max_delay = max_delay if max_delay is not None else (cfg.max_delay if cfg is not None else None)
        self.seed = seed if seed is not None else (cfg.seed if cfg is not None else None)
        self.overlap = overlap and self.max_delay is not None and self.seed is not None
        if delay is None and self.overlap:
            from . import binding

            delay = lambda step, sender, receiver: binding.tensair_delay(self.seed, self.max_delay, step, sender, receiver)
        self._delay = delay
        self._lane = None
        self._flying = {}            # (sender, step) -> [completion token, first step needed here, bytes received]
        self.bytes_sent = 0
        self.bytes_received = 0
        self.bytes_waited_at_own_step = 0     # received bytes the training stream had to wait for in the step they were sent
        self.bytes_waited_later = 0           # received bytes that travelled while later batches were trained

    # ------------------------------------------------------------------ helpers
    def _global_rank(self, group_rank: int) -> int:
        return group_rank if self.group is None else self.dist.get_global_rank(self.group, group_rank)

    def _is_local(self, g: int) -> bool:
        return self.first <= g < self.first + self.local

    def _lane_for(self, sample_tensor):
        if self._lane is None:
            if sample_tensor.is_cuda:
                import torch

                main = getattr(self.port, "stream", None) or torch.cuda.current_stream(sample_tensor.device)
                self._lane = _CudaLane(torch, main)
            else:
                self._lane = _HostLane()
        return self._lane

    def first_needed(self, sender: int, step: int) -> int:
        """The first step at whose apply call a replica held here needs the message of (sender, step)."""
        if not self.overlap:
            return step
        delays = [self._delay(step, sender, j) for j in range(self.first, self.first + self.local) if j != sender]
        return step + (min(delays) if delays else self.max_delay)

    def _row_counts(self, step: int, lane, torch):
        """[process][local replica] -> (rows, input rows) of every message of `step`."""
        header = getattr(self.port, "tensair_message_header", None)
        with lane.run():
            if header is not None:
                # the counts are read where the kernels left them, on the communication stream: the training stream
                # is not synchronised
                mine = torch.stack([header(self.first + r, step)[:2] for r in range(self.local)]).to(torch.int64)
                if mine.device.type != torch.device(self.count_device).type:
                    mine = mine.to(self.count_device)
            else:
                mine = torch.tensor([self.port.tensair_message_rows(r, step) for r in range(self.local)],
                                    dtype=torch.int64, device=self.count_device).reshape(self.local, 2)
            gathered = [torch.empty_like(mine) for _ in range(self.world_size)]
            self.dist.all_gather(gathered, mine, group=self.group)
            stacked = torch.stack(gathered)
            if stacked.is_cuda:
                host = torch.empty(stacked.shape, dtype=stacked.dtype, pin_memory=True)
                host.copy_(stacked, non_blocking=True)
                lane.host_wait([])
                stacked = host
        return stacked.tolist()

    # ------------------------------------------------------------------ the step
    def exchange(self, step: int):
        """After the local train calls of `step`: starts the transfer of every message of that step (this process's
        out, the others' into this process's pool) and files the received ones.  Collective: every process calls it
        for every step.  It returns once the transfers are enqueued; apply() waits for what it needs."""
        import torch

        if self.world_size == 1:
            return
        if self.dist is None:
            raise RuntimeError("exchange() between processes needs torch.distributed")
        probe = self.port.tensair_message_buffers(self.first, step)[0]
        lane = self._lane_for(probe)
        lane.begin()
        rows = self._row_counts(step, lane, torch)
        for g in range(self.world_replicas):
            owner, r = divmod(g, self.local)
            n, n_in = rows[owner][r]
            ids, delta = self.port.tensair_message_buffers(g, step)
            stride = delta.numel() // ids.numel()
            requests = []
            with lane.run():
                if n:
                    src = self._global_rank(owner)
                    for part in (ids[:n], delta[:n * stride]):
                        req = self.dist.broadcast(part, src=src, group=self.group, async_op=lane.async_op)
                        if lane.async_op:
                            requests.append(req)
                moved = n * (4 + 4 * stride)
                if owner == self.rank:
                    self.bytes_sent += moved * (self.world_size - 1)
                    received = 0
                else:
                    self.bytes_received += moved
                    received = moved
                    # filed at once and in the one-process order; the slot's header and index are written behind the
                    # rows on the communication stream
                    if lane.commit_stream is not None:
                        self.port.tensair_commit_message(g, step, n, n_in, stream=lane.commit_stream)
                    else:
                        self.port.tensair_commit_message(g, step, n, n_in)
                self._flying[(g, step)] = [lane.mark(requests), self.first_needed(g, step), received]

    def _wait_for(self, key, at_step: int):
        token, _, received = self._flying.pop(key)
        self._lane.stream_wait(token)
        if received:
            if key[1] == at_step:
                self.bytes_waited_at_own_step += received
            else:
                self.bytes_waited_later += received

    def apply(self, step: int) -> int:
        """Gradient application of what is due at `step`: for real on the replicas held here, as book-keeping
        for the others.  The training stream first waits for the messages that are due here now (and no others).
        Returns the messages applied to local replicas."""
        for key in sorted(k for k, v in self._flying.items() if v[1] <= step and not self._is_local(k[0])):
            self._wait_for(key, step)
        applied = self.port.tensair_apply_step(step)          # all local replicas in one pass over their tables
        for g in range(self.world_replicas):
            if not self._is_local(g):
                self.port.tensair_shadow_apply(g, step, False)
        # The next batches reuse the pool slots of step - max_delay: what was sent from them must have left.
        horizon = step - (self.max_delay if self.max_delay is not None else 0)
        for key in sorted(k for k in self._flying if k[1] <= horizon):
            self._wait_for(key, step)
        return applied

    def drain(self) -> int:
        for key in sorted(self._flying):
            self._wait_for(key, -1)
        return self.port.tensair_drain()

    def hidden_share(self) -> float:
        """Of the bytes received so far and waited for, the share that travelled while later batches were trained."""
        total = self.bytes_waited_at_own_step + self.bytes_waited_later
        return self.bytes_waited_later / total if total else 0.0

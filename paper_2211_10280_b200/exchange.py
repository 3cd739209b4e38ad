"""Replicas spread over processes, one GPU each: the message exchange between them.

The paper places one Model instance per worker and has each send its gradient to every other instance
(Section 2.2, data parallelism; Algorithm 1, send_gradients).  Here a job of `world_size` processes holds
`local` replicas each (global id = rank * local + local index).  Per step every process trains its own
replicas, then the messages travel: each sender announces its row counts (one small all-gather), and its
row ids and delta rows are broadcast straight out of its pool slot into the slot the other processes keep
for that sender - no staging copy, no padding to a common size.  After that every process holds every
message in its own GPU memory and applies what is due with the same kernels as a one-process job; the
delivery schedule is a function of the seed, so every process keeps the whole of it and the result is the
one-process result bit for bit.

Only plumbing lives here (torch.distributed calls and the order of the library calls); the arithmetic is
the library's.  `port` is a binding.Context created with world_replicas / first_replica, or anything with
the same calls (the CPU tests use a stand-in that needs no GPU).
"""
from __future__ import annotations


class ShardedReplicas:
    def __init__(self, port, rank: int, world_size: int, local: int, dist=None, group=None, count_device="cpu"):
        """dist: torch.distributed (initialised); may be None when world_size == 1 or when the caller moves the
        messages itself and uses only apply() and drain().  count_device: where the small tensor of row counts
        lives for the all-gather ("cuda" with nccl, "cpu" with gloo)."""
        self.port, self.rank, self.world_size, self.local = port, rank, world_size, local
        self.dist, self.group, self.count_device = dist, group, count_device
        self.world_replicas = world_size * local
        self.first = rank * local
        self.bytes_sent = 0
        self.bytes_received = 0

    def _global_rank(self, group_rank: int) -> int:
        return group_rank if self.group is None else self.dist.get_global_rank(self.group, group_rank)

    def exchange(self, step: int):
        """After the local train calls of `step`: brings every other process's messages of that step into
        this process's pool and files them.  Collective: every process calls it for every step."""
        import torch

        if self.world_size == 1:
            return
        if self.dist is None:
            raise RuntimeError("exchange() between processes needs torch.distributed")
        mine = [self.port.tensair_message_rows(r, step) for r in range(self.local)]
        counts = torch.tensor(mine, dtype=torch.int64, device=self.count_device).reshape(self.local, 2)
        gathered = [torch.empty_like(counts) for _ in range(self.world_size)]
        self.dist.all_gather(gathered, counts, group=self.group)
        rows = torch.stack(gathered).cpu().tolist()           # [process][local replica] -> (rows, input rows)
        for g in range(self.world_replicas):
            owner, r = divmod(g, self.local)
            n, n_in = rows[owner][r]
            ids, delta = self.port.tensair_message_buffers(g, step)
            stride = delta.numel() // ids.numel()
            if n:
                src = self._global_rank(owner)
                self.dist.broadcast(ids[:n], src=src, group=self.group)
                self.dist.broadcast(delta[:n * stride], src=src, group=self.group)
            moved = n * (4 + 4 * stride)
            if owner == self.rank:
                self.bytes_sent += moved * (self.world_size - 1)
            else:
                self.bytes_received += moved
                self.port.tensair_commit_message(g, step, n, n_in)

    def apply(self, step: int) -> int:
        """Gradient application of what is due at `step`: for real on the replicas held here, as book-keeping
        for the others.  Returns the messages applied to local replicas."""
        applied = self.port.tensair_apply_step(step)          # all local replicas in one pass over their tables
        for g in range(self.world_replicas):
            if not self.first <= g < self.first + self.local:
                self.port.tensair_shadow_apply(g, step, False)
        return applied

    def drain(self) -> int:
        return self.port.tensair_drain()

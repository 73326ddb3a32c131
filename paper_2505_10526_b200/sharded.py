"""Acceptance with the LM head's vocabulary cut across ranks (tensor-parallel targets).

Every arithmetic step is a ``massv_shard_*`` kernel call; this module only owns the buffers and moves the
three small exchange buffers between ranks (three all-gathers per step, one at temperature 0).
``ShardedAccept`` is one rank.  The exchange is either of:

* ``DistComm``  -- ``torch.distributed`` collectives (NCCL between GPUs; gloo in the CPU tests);
* ``run_lockstep`` -- all ranks of a world on ONE device, phase by phase, concatenation in place of the
  all-gather: the single-GPU check of the multi-rank path (no rank's kernel waits on another's).  Its
  "publish" transport uses the library's own all-gather-by-stores kernel (``massv_shard_publish``), the
  ranks' gathered buffers standing for peer-mapped memory.

The phases are a generator's steps: a rank yields the buffer it wants gathered and is resumed with the
gathered one, so both transports drive the same code.
"""
from __future__ import annotations

import torch

from . import binding as mv


class DistComm:
    """All-gather over a ``torch.distributed`` process group (ranks in order = vocabulary order)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        """[n] on every rank -> [world * n], rank r's copy at r * n."""
        out = torch.empty((self.world * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        self.dist.all_gather_into_tensor(out, t.contiguous(), group=self.group)
        return out


def drive(phases, comm):
    """Run one rank's phase generator against a communicator."""
    try:
        t = next(phases)
        while True:
            t = phases.send(comm.all_gather(t))
    except StopIteration as e:
        return e.value


def run_lockstep(ranks, inputs, transport="concat"):
    """All ranks on one device: advance every rank to its next exchange, combine, resume.
    ``ranks``: list of ShardedAccept in rank order; ``inputs``: per-rank kwargs of ``phases``.
    ``transport``: "concat" (concatenation stands for the collective) or "publish" (every rank stores its
    buffer into every rank's gathered buffer with ``massv_shard_publish``; stream order on the one device
    stands for the barrier between publishing and reading)."""
    gens = [r.phases(**kw) for r, kw in zip(ranks, inputs)]
    reqs = [next(g) for g in gens]
    while True:
        if transport == "publish":
            world = len(reqs)
            bufs = [torch.empty((world * t.numel(),), dtype=t.dtype, device=t.device) for t in reqs]
            for r, t in enumerate(reqs):
                mv.massv_shard_publish(t, bufs, r)
        else:
            cat = torch.cat(reqs, dim=0)
            bufs = [cat.clone() for _ in reqs]
        nxt, done = [], []
        for g, buf in zip(gens, bufs):
            try:
                nxt.append(g.send(buf))
            except StopIteration as e:
                done.append(e.value)
        if done:
            assert len(done) == len(gens), "ranks finished at different phases"
            return done
        reqs = nxt


class ShardedAccept:
    """One rank's buffers and call sequence for a fixed (batch, gamma, hidden, shard size, temperature)."""

    def __init__(self, batch, gamma, hidden, vocab_shard, temperature, world, rank, device="cuda"):
        self.desc = mv.accept_desc(batch, gamma, hidden, vocab_shard, temperature)
        self.B, self.g, self.Vs, self.T = batch, gamma, vocab_shard, float(temperature)
        self.world, self.rank = world, rank
        M = batch * (gamma + 1)
        dev = torch.device(device)
        f32, i32 = torch.float32, torch.int32
        words = mv.massv_shard_stats_words(self.desc)
        if words == 0:
            raise mv.MassvError(-2, "massv_shard_stats_words")
        self.stats = torch.empty((words,), dtype=f32, device=dev)
        self.logits = torch.empty((M, vocab_shard), dtype=f32, device=dev) if temperature > 0 else None
        self.state = torch.empty((mv.massv_shard_state_bytes(self.desc),), dtype=torch.uint8, device=dev)
        self.masses = torch.empty((mv.massv_shard_mass_count(self.desc),), dtype=torch.float64, device=dev)
        self.token = torch.empty((batch,), dtype=i32, device=dev)
        self.out_tokens = torch.empty((batch, gamma + 1), dtype=i32, device=dev)
        self.accept_len = torch.empty((batch,), dtype=i32, device=dev)
        self.dev_status = torch.zeros((1,), dtype=i32, device=dev)
        self.marks = None           # set to a list to collect (name, CUDA event) pairs around the kernel calls

    def _mark(self, name):
        if self.marks is not None:
            e = torch.cuda.Event(enable_timing=True)
            e.record()
            self.marks.append((name, e))

    def phases(self, hidden, lm_head_shard, draft_tokens, draft_probs_shard=None, u_accept=None, u_sample=None):
        """Generator: yields a buffer to all-gather, is resumed with the gathered one."""
        d, W, r, st = self.desc, self.world, self.rank, self.dev_status
        sampling = self.T > 0
        self._mark("lm_head:start")
        n = mv.massv_shard_lm_head(d, W, r, hidden, lm_head_shard, self.logits, self.stats, st)
        if sampling:
            mv.massv_shard_gather_draft(d, W, r, self.logits, draft_probs_shard, draft_tokens, self.stats, st)
        self._mark("lm_head:stop")
        stats_all = yield self.stats
        self._mark("scan:start")
        mv.massv_shard_scan(d, W, n, stats_all, draft_tokens, u_accept, self.out_tokens, self.accept_len, self.state, st)
        if sampling:
            mv.massv_shard_masses(d, W, r, self.logits, draft_probs_shard, self.state, self.masses, st)
            self._mark("scan:stop")
            masses_all = yield self.masses
            self._mark("pick:start")
            mv.massv_shard_pick(d, W, r, masses_all, u_sample, self.state, self.logits, draft_probs_shard,
                                self.token, st)
            self._mark("pick:stop")
            tokens_all = yield self.token
            self._mark("set_token:start")
            mv.massv_shard_set_token(d, W, self.state, tokens_all, self.out_tokens, st)
            self._mark("set_token:stop")
        else:
            self._mark("scan:stop")
        return self.out_tokens, self.accept_len

    def run(self, comm, **inputs):
        """One step of this rank against a communicator (every rank of the group calls it)."""
        return drive(self.phases(**inputs), comm)

"""Acceptance with the LM head's vocabulary cut across ranks (tensor-parallel targets).

Every arithmetic step is a ``massv_shard_*`` kernel call; this module only owns the buffers and moves the
three small gathered arrays between ranks.  ``ShardedAccept`` is one rank.  The exchange is a ``Comm``:

* ``DistComm``  -- ``torch.distributed`` collectives (NCCL between GPUs; gloo in the CPU tests);
* ``run_lockstep`` -- all ranks of a world on ONE device, phase by phase, concatenation in place of the
  all-gather: the single-GPU check of the multi-rank path (no rank's kernel waits on another's).

The phases are generators' steps: each rank yields what it wants gathered / reduced and is resumed with
the result, so both transports drive the same code.
"""
from __future__ import annotations

import torch

from . import binding as mv


class DistComm:
    """Collectives over a ``torch.distributed`` process group (ranks in order = vocabulary order)."""

    def __init__(self, group=None):
        import torch.distributed as dist
        self.dist, self.group = dist, group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)

    def all_gather(self, t: torch.Tensor) -> torch.Tensor:
        """[n, ...] on every rank -> [world * n, ...], rank-major."""
        out = torch.empty((self.world * t.shape[0],) + tuple(t.shape[1:]), dtype=t.dtype, device=t.device)
        self.dist.all_gather_into_tensor(out, t.contiguous(), group=self.group)
        return out

    def all_reduce_max(self, t: torch.Tensor) -> torch.Tensor:
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX, group=self.group)
        return t


def drive(phases, comm):
    """Run one rank's phase generator against a communicator."""
    try:
        kind, t = next(phases)
        while True:
            res = comm.all_gather(t) if kind == "gather" else comm.all_reduce_max(t)
            kind, t = phases.send(res)
    except StopIteration as e:
        return e.value


def run_lockstep(ranks, inputs):
    """All ranks on one device: advance every rank to its next exchange, combine, resume.
    ``ranks``: list of ShardedAccept in rank order; ``inputs``: per-rank kwargs of ``phases``."""
    gens = [r.phases(**kw) for r, kw in zip(ranks, inputs)]
    reqs = [next(g) for g in gens]
    while True:
        kinds = {k for k, _ in reqs}
        assert len(kinds) == 1, "ranks disagree on the exchange"
        if kinds == {"gather"}:
            res = [torch.cat([t for _, t in reqs], dim=0)] * len(gens)
        else:
            m = torch.stack([t for _, t in reqs], dim=0).amax(dim=0)
            res = [m.clone() for _ in gens]
        nxt, done = [], []
        for g, r in zip(gens, res):
            try:
                nxt.append(g.send(r))
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
        slots = mv.massv_shard_max_partials(self.desc)
        if slots == 0:
            raise mv.MassvError(-2, "massv_shard_max_partials")
        self.part_max = torch.empty((slots, M), dtype=f32, device=dev)
        self.part_sum = torch.empty((slots, M), dtype=f32, device=dev)
        self.part_idx = torch.empty((slots, M), dtype=i32, device=dev)
        self.logits = torch.empty((M, vocab_shard), dtype=f32, device=dev) if temperature > 0 else None
        self.z_at = torch.empty((batch, gamma), dtype=f32, device=dev)
        self.q_at = torch.empty((batch, gamma), dtype=f32, device=dev)
        self.state = torch.empty((mv.massv_shard_state_bytes(self.desc),), dtype=torch.uint8, device=dev)
        n_chunks = mv.massv_shard_chunks(self.desc)
        self.mass_res = torch.empty((1, batch, n_chunks), dtype=torch.float64, device=dev)
        self.mass_p = torch.empty((1, batch, n_chunks), dtype=torch.float64, device=dev)
        self.token = torch.empty((batch,), dtype=i32, device=dev)
        self.out_tokens = torch.empty((batch, gamma + 1), dtype=i32, device=dev)
        self.accept_len = torch.empty((batch,), dtype=i32, device=dev)
        self.dev_status = torch.zeros((1,), dtype=i32, device=dev)

    def phases(self, hidden, lm_head_shard, draft_tokens, draft_probs_shard=None, u_accept=None, u_sample=None):
        d, W, r, st = self.desc, self.world, self.rank, self.dev_status
        sampling = self.T > 0
        n = mv.massv_shard_lm_head(d, W, r, hidden, lm_head_shard, self.logits, self.part_max, self.part_sum,
                                   self.part_idx, st)
        if sampling and self.g > 0:
            mv.massv_shard_gather_draft(d, W, r, self.logits, draft_probs_shard, draft_tokens, self.z_at, self.q_at, st)
            z_at = yield ("max", self.z_at)
            q_at = yield ("max", self.q_at)
        else:
            z_at = q_at = None
        pm = yield ("gather", self.part_max[:n])
        ps = yield ("gather", self.part_sum[:n])
        pi = yield ("gather", self.part_idx[:n])
        mv.massv_shard_scan(d, W, pm.shape[0], pm, ps, pi, draft_tokens, z_at, q_at, u_accept, self.out_tokens,
                            self.accept_len, self.state, st)
        if sampling:
            mv.massv_shard_masses(d, W, r, self.logits, draft_probs_shard, self.state, self.mass_res, self.mass_p, st)
            res_all = yield ("gather", self.mass_res)
            p_all = yield ("gather", self.mass_p)
            mv.massv_shard_pick(d, W, r, res_all, p_all, u_sample, self.state, self.logits, draft_probs_shard,
                                self.token, st)
            tok = yield ("max", self.token)
            mv.massv_shard_set_token(d, self.state, tok, self.out_tokens, st)
        return self.out_tokens, self.accept_len

    def run(self, comm, **inputs):
        """One step of this rank against a communicator (every rank of the group calls it)."""
        return drive(self.phases(**inputs), comm)

"""Acceptance with the LM head's vocabulary cut across ranks (tensor-parallel targets).

Every arithmetic step is a ``massv_shard_*`` kernel call; this module only owns the buffers and moves the
three small exchange buffers between ranks (three all-gathers per step, one at temperature 0).
``ShardedAccept`` is one rank.  The exchange is either of:

* ``DistComm``  -- ``torch.distributed`` collectives (NCCL between GPUs; gloo in the CPU tests);
* ``run_lockstep`` -- all ranks of a world on ONE device, phase by phase, concatenation in place of the
  all-gather: the single-GPU check of the multi-rank path (no rank's kernel waits on another's).  Its
  "publish" transport uses the library's own all-gather-by-stores kernel (``massv_shard_publish``), the
  ranks' gathered buffers standing for peer-mapped memory.  ``python -m paper_2505_10526_b200.sharded
  --config NAME --world W`` runs it on a named workload and prints rank 0's kernel times.

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


def _main():
    """All ranks of a world on one GPU, in lockstep, on a named synthetic workload: checks that the ranks
    agree and prints one JSON line with rank 0's kernel times per phase (medians; the exchanges between
    the phases are not in them) and the bytes each rank contributes to every exchange."""
    import argparse
    import json

    from workloads import generate, get_config

    ap = argparse.ArgumentParser(description=_main.__doc__)
    ap.add_argument("--config", default="qwen7b_b16_t1")
    ap.add_argument("--world", type=int, default=4)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--transport", choices=["concat", "publish"], default="publish")
    a = ap.parse_args()
    cfg = get_config(a.config)
    if cfg.vocab % a.world:
        raise SystemExit("the vocabulary must divide evenly among the ranks")
    w = generate(cfg, device="cuda", with_attention=False)
    Vs = cfg.vocab // a.world
    ranks = [ShardedAccept(cfg.batch, cfg.gamma, cfg.hidden, Vs, cfg.temperature, a.world, r) for r in range(a.world)]
    inputs = []
    for r in range(a.world):
        kw = dict(hidden=w["hidden"], lm_head_shard=w["lm_head"][r * Vs:(r + 1) * Vs].contiguous(),
                  draft_tokens=w["draft_tokens"])
        if cfg.temperature > 0:
            kw.update(draft_probs_shard=w["draft_probs"][:, :, r * Vs:(r + 1) * Vs].contiguous(),
                      u_accept=w["u_accept"], u_sample=w["u_sample"])
        inputs.append(kw)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")       # larger than L2
    spans = {}
    for it in range(a.warmup + a.iters):
        flush.zero_()
        ranks[0].marks = [] if it >= a.warmup else None
        res = run_lockstep(ranks, inputs, transport=a.transport)
        torch.cuda.synchronize()
        for t, l in res[1:]:
            assert torch.equal(t, res[0][0]) and torch.equal(l, res[0][1]), "ranks disagree"
        if ranks[0].marks:
            ev = dict(ranks[0].marks)
            for name in ("lm_head", "scan", "pick", "set_token"):
                if name + ":start" in ev:
                    spans.setdefault(name, []).append(ev[name + ":start"].elapsed_time(ev[name + ":stop"]))
    assert all(int(r.dev_status.item()) == 0 for r in ranks)
    med = {k: round(sorted(v)[len(v) // 2], 4) for k, v in spans.items()}
    r0 = ranks[0]
    print(json.dumps(dict(workload=cfg.name, world=a.world, transport=a.transport, shard_vocab=Vs,
                          rank0_kernel_ms=med, rank0_kernel_ms_total=round(sum(med.values()), 4),
                          exchange_bytes_per_rank=dict(stats=r0.stats.numel() * 4, masses=r0.masses.numel() * 8,
                                                       token=r0.token.numel() * 4),
                          mean_accept_len=float(res[0][1].float().mean()))))


if __name__ == "__main__":
    _main()

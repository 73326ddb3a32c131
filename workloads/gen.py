"""Seeded generator for verify-step inputs.

Every tensor is drawn from one ``torch.Generator`` seeded with the config's
seed, in a fixed order, on the requested device (the CPU generator and the CUDA
generator give different streams; each is reproducible on its own), except the
uniforms of the acceptance tests and of the draw: those come from Philox4x32-10
keyed by the seed (workloads/philox.py) and are the same on either device.
Values destined for bf16 tensors are drawn in fp32 and rounded once
(round-to-nearest-even), so every consumer sees the same bf16 bits.

The draft distribution q and the drafted tokens are *inputs* of the verify
step.  They are built here from the target's own logits plus Gaussian noise
with library matmul / softmax calls in fp32; nothing under test is used.
"""
from __future__ import annotations

import math

import torch

from . import philox
from .configs import VerifyConfig

PAGE_SIZE = 16


def _randn_bf16(shape, std, gen, device, chunk_rows=16384):
    """N(0, std) in fp32 rounded to bf16, generated in row chunks to bound memory."""
    out = torch.empty(shape, dtype=torch.bfloat16, device=device)
    flat = out.view(shape[0], -1)
    for r0 in range(0, shape[0], chunk_rows):
        r1 = min(shape[0], r0 + chunk_rows)
        blk = torch.randn((r1 - r0, flat.shape[1]), generator=gen, device=device, dtype=torch.float32)
        if std != 1.0:
            blk.mul_(std)
        flat[r0:r1] = blk.to(torch.bfloat16)
    return out


def kv_bytes(cfg: VerifyConfig, seq_lens) -> int:
    """Bytes of K and V that one verify step must read: every cached position
    plus the gamma+1 appended ones, once each, for every KV head."""
    w = getattr(cfg, "window", 0)
    tot = int(sum(min(int(l) + cfg.rows, w + cfg.rows - 1) if w > 0 else int(l) + cfg.rows for l in seq_lens))
    return tot * cfg.n_kv_heads * cfg.head_dim * 2 * 2


def generate(cfg: VerifyConfig, device="cpu", with_lm_head=True, with_attention=True):
    """Return a dict of tensors for one verify step of ``cfg`` on ``device``.

    Attention side
      q        bf16 [B, R, Hq, d]      queries of the R = gamma+1 block rows
      k_new    bf16 [B, R, Hkv, d]     block keys / values to append at L_b .. L_b+gamma
      v_new
      k_pages  bf16 [P, Hkv, 16, d]    page pool (random page ids per sequence)
      v_pages
      page_table int32 [B, max_pages]  -1 where unmapped
      seq_lens int32 [B]               committed length L_b before the step
      n_image  int32 [B]               leading image tokens (metadata only)
    Acceptance side
      hidden   bf16 [B, R, K]; lm_head bf16 [V, K]
      draft_tokens int32 [B, gamma]
      draft_probs  fp32 [B, gamma, V]  (T > 0 only)
      u_accept fp32 [B, gamma], u_sample fp32 [B, R]  in [0, 1)
    """
    dev = torch.device(device)
    gen = torch.Generator(device=dev)
    gen.manual_seed(cfg.seed)
    B, R, g = cfg.batch, cfg.rows, cfg.gamma
    out = {}

    # context lengths (drawn even when attention tensors are skipped so that
    # the remaining stream does not depend on the flags)
    if cfg.ctx_lo == cfg.ctx_hi:
        seq = torch.full((B,), cfg.ctx_lo, dtype=torch.int64)
    else:
        seq = torch.randint(cfg.ctx_lo, cfg.ctx_hi + 1, (B,), generator=gen, device=dev).cpu()
    if cfg.image_tokens >= 1:
        n_img = torch.minimum(seq, torch.tensor(int(cfg.image_tokens)))
    else:
        n_img = (seq.double() * cfg.image_tokens).floor().long()
    out["seq_lens"] = seq.to(torch.int32).to(dev)
    out["n_image"] = n_img.to(torch.int32).to(dev)

    if with_attention:
        pages_per_seq = [(int(l) + R + PAGE_SIZE - 1) // PAGE_SIZE for l in seq]
        max_pages = max(pages_per_seq)
        n_pages = sum(pages_per_seq) + 3            # a few never-mapped pages stay in the pool
        perm = torch.randperm(n_pages, generator=gen, device=dev).cpu()
        table = torch.full((B, max_pages), -1, dtype=torch.int32)
        off = 0
        for b, n in enumerate(pages_per_seq):
            table[b, :n] = perm[off:off + n].to(torch.int32)
            off += n
        out["page_table"] = table.to(dev)
        Hq, Hkv, d = cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim
        out["k_pages"] = _randn_bf16((n_pages, Hkv, PAGE_SIZE, d), 1.0, gen, dev, chunk_rows=4096)
        out["v_pages"] = _randn_bf16((n_pages, Hkv, PAGE_SIZE, d), 1.0, gen, dev, chunk_rows=4096)
        out["q"] = _randn_bf16((B, R, Hq, d), 1.0, gen, dev)
        out["k_new"] = _randn_bf16((B, R, Hkv, d), 1.0, gen, dev)
        out["v_new"] = _randn_bf16((B, R, Hkv, d), 1.0, gen, dev)

    if with_lm_head:
        K, V = cfg.hidden, cfg.vocab
        out["hidden"] = _randn_bf16((B, R, K), cfg.hidden_std, gen, dev)
        out["lm_head"] = _randn_bf16((V, K), 0.02, gen, dev)
        # the drafter: target logits (library fp32 matmul) + N(0, noise_std)
        h32 = out["hidden"].view(B * R, K).float()
        z = torch.empty((B * R, V), dtype=torch.float32, device=dev)
        step = 32768
        for v0 in range(0, V, step):
            z[:, v0:v0 + step] = h32 @ out["lm_head"][v0:v0 + step].float().t()
        z = z.view(B, R, V)[:, :g]                   # drafter rows: positions t+1 .. t+gamma
        noise = torch.randn(z.shape, generator=gen, device=dev, dtype=torch.float32)
        zq = z + cfg.draft_noise_std * noise
        del noise
        if cfg.temperature > 0:
            qprob = torch.softmax(zq / cfg.temperature, dim=-1).contiguous()
            tok = torch.multinomial(qprob.view(B * g, V), 1, generator=gen).view(B, g)
            out["draft_probs"] = qprob
        else:
            tok = zq.argmax(dim=-1)
        out["draft_tokens"] = tok.to(torch.int32).contiguous()
        # the uniforms of the rejection tests and of the draw: Philox4x32-10 keyed by the config's seed, so the
        # same numbers on either device (stream 0: acceptance, stream 1: draw)
        out["u_accept"] = torch.from_numpy(philox.uniforms(B * g, cfg.seed, 0)).view(B, g).to(dev)
        out["u_sample"] = torch.from_numpy(philox.uniforms(B * R, cfg.seed, 1)).view(B, R).to(dev)
    return out

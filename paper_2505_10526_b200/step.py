"""One verify step = massv_verify_attn + massv_accept + massv_kv_commit.

``VerifyStep`` owns the descriptors, the scratch buffers and the output tensors
for a fixed geometry, so that a step is three C-ABI calls and nothing else.  All
arithmetic happens inside ``libmassv.so``.
"""
from __future__ import annotations

import torch

from . import binding as mv

# tensors that change every step (the rest - page pools, page table, lengths,
# LM-head weights - is resident state)
STEP_INPUTS = ("q", "k_new", "v_new", "hidden", "draft_tokens", "draft_probs", "u_accept", "u_sample")


class VerifyStep:
    def __init__(self, batch, gamma, n_q_heads, n_kv_heads, head_dim, hidden, vocab, temperature,
                 max_pages_per_seq, num_pages, device="cuda", kv_chunk=0, scale=0.0, window=0,
                 attn_kernel=0, want_logits=False, want_probs=False, want_attn_f32=False):
        self.device = torch.device(device)
        self.B, self.gamma, self.R = batch, gamma, gamma + 1
        self.T = float(temperature)
        self.adesc = mv.attn_desc(batch, gamma, n_q_heads, n_kv_heads, head_dim, max_pages_per_seq, num_pages,
                                  scale=scale, kv_chunk=kv_chunk, window=window, kernel=attn_kernel)
        self.cdesc = mv.accept_desc(batch, gamma, hidden, vocab, temperature)
        dev = self.device
        self.attn_ws = mv.alloc_workspace(mv.massv_verify_attn_workspace_size(self.adesc), dev)
        self.accept_ws = mv.alloc_workspace(mv.massv_accept_workspace_size(self.cdesc), dev)
        self.attn_out = torch.empty((batch, self.R, n_q_heads, head_dim), dtype=torch.bfloat16, device=dev)
        self.attn_out_f32 = torch.empty_like(self.attn_out, dtype=torch.float32) if want_attn_f32 else None
        self.lse = torch.empty((batch, self.R, n_q_heads), dtype=torch.float32, device=dev) if want_attn_f32 else None
        # tokens and accepted lengths share one buffer, so that a host reads both back with one copy
        self._out_blob = torch.empty((batch * self.R + batch,), dtype=torch.int32, device=dev)
        self.out_tokens = self._out_blob[:batch * self.R].view(batch, self.R)
        self.accept_len = self._out_blob[batch * self.R:]
        self.logits = torch.empty((batch, self.R, vocab), dtype=torch.float32, device=dev) if want_logits else None
        self.probs = (torch.empty((batch, self.R, vocab), dtype=torch.float32, device=dev)
                      if want_probs and temperature > 0 else None)
        self.dev_status = torch.zeros((1,), dtype=torch.int32, device=dev)
        self._staging = None
        self._host_out = None

    @classmethod
    def for_workload(cls, cfg, w, **kw):
        return cls(cfg.batch, cfg.gamma, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.hidden, cfg.vocab,
                   cfg.temperature, w["page_table"].shape[1], w["k_pages"].shape[0],
                   device=w["k_pages"].device, **{"window": getattr(cfg, "window", 0), **kw})

    # -- the three calls -------------------------------------------------------------
    def attn(self, w):
        mv.massv_verify_attn(self.adesc, w["q"], w["k_new"], w["v_new"], w["k_pages"], w["v_pages"],
                             w["page_table"], w["seq_lens"], self.attn_out, self.attn_out_f32, self.lse,
                             self.attn_ws, self.dev_status)

    def accept(self, w):
        sampling = self.T > 0
        mv.massv_accept(self.cdesc, w["hidden"], w["lm_head"], w["draft_tokens"],
                        w.get("draft_probs") if sampling else None, w.get("u_accept") if sampling else None,
                        w.get("u_sample") if sampling else None, self.out_tokens, self.accept_len,
                        self.logits, self.probs, self.accept_ws, self.dev_status)

    def commit(self, seq_lens, rollback=False):
        mv.massv_kv_commit(self.B, self.gamma, None if rollback else self.accept_len, seq_lens, self.dev_status)

    def run(self, w, commit=True):
        """Enqueue one whole step on the current stream (no synchronisation)."""
        self.attn(w)
        self.accept(w)
        if commit:
            self.commit(w["seq_lens"])

    # -- end-to-end step with host buffers ----------------------------------------------
    def host_inputs_like(self, tensors):
        """Pinned host buffers for per-step inputs, shaped like ``tensors`` (a dict of name ->
        tensor): a ``HostInputs`` dict whose values are views of ONE pinned allocation, mirrored by
        ONE device allocation, so that ``run_host`` moves a step's inputs with a single copy however
        many tensors they are.  The caller writes each step's inputs into the returned views in place.
        Several sets may exist side by side (say, one with and one without the draft distributions)."""
        return HostInputs(tensors, self.device)

    def _host_result(self):
        if self._host_out is None:
            self._host_out_blob = torch.empty(self._out_blob.shape, dtype=torch.int32).pin_memory()
            n_tok = self.B * self.R
            self._host_out = (self._host_out_blob[:n_tok].view(self.B, self.R), self._host_out_blob[n_tok:])
        return self._host_out

    def run_host(self, host_inputs, resident, commit=False):
        """One step whose per-step inputs start in pinned host memory and whose result (tokens and
        accepted lengths) ends in pinned host memory.  ``host_inputs`` is what ``host_inputs_like``
        returned (one copy up, one copy down) or any dict of pinned tensors (one copy per tensor);
        ``resident`` holds everything that already lives on the device.  Returns (out_tokens,
        accept_len) host tensors after synchronising."""
        w = dict(resident)
        out = self._host_result()
        if isinstance(host_inputs, HostInputs):
            host_inputs.dev_blob.copy_(host_inputs.host_blob, non_blocking=True)
            w.update(host_inputs.dev_views)
        else:
            if self._staging is None or set(self._staging) != set(host_inputs):
                self._staging = {k: torch.empty_like(v, device=self.device) for k, v in host_inputs.items()}
            for k, v in host_inputs.items():
                self._staging[k].copy_(v, non_blocking=True)
                w[k] = self._staging[k]
        self.run(w, commit=commit)
        self._host_out_blob.copy_(self._out_blob, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return out

    def host_bytes_per_step(self, host_inputs):
        if isinstance(host_inputs, HostInputs):
            h2d = host_inputs.host_blob.numel()     # the whole staging buffer goes up, padding included
        else:
            h2d = sum(v.numel() * v.element_size() for v in host_inputs.values())
        d2h = self.out_tokens.numel() * 4 + self.accept_len.numel() * 4
        return h2d, d2h


class HostInputs(dict):
    """name -> pinned host view; ``host_blob`` / ``dev_blob`` are the two allocations behind the
    views and ``dev_views`` the device-side tensors of the same names."""

    def __init__(self, tensors, device, align=256):
        layout, off = {}, 0
        for k, v in tensors.items():
            nbytes = v.numel() * v.element_size()
            layout[k] = (off, nbytes, v.dtype, tuple(v.shape))
            off = (off + nbytes + align - 1) // align * align
        self.host_blob = torch.empty((max(off, align),), dtype=torch.uint8).pin_memory()
        self.dev_blob = torch.empty((max(off, align),), dtype=torch.uint8, device=device)
        view = lambda blob: {k: blob[o:o + n].view(dt).view(shape) for k, (o, n, dt, shape) in layout.items()}
        super().__init__(view(self.host_blob))
        self.dev_views = view(self.dev_blob)
        for k, v in tensors.items():
            self[k].copy_(v)

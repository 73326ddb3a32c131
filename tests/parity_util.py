"""Helpers that compare the CUDA path's outputs with the CPU oracle's."""
from __future__ import annotations

import numpy as np
import torch

import oracle

MARGIN = 1e-3          # decisions whose oracle margin is below this may differ (counted, reported)
TIGHT = 1e-6


def sub_workload(w, idx):
    """Workload restricted to the sequences in idx (page pools and LM head stay whole)."""
    idx_t = torch.as_tensor(idx, device=w["seq_lens"].device, dtype=torch.long)
    out = {}
    for k, v in w.items():
        if k in ("k_pages", "v_pages", "lm_head"):
            out[k] = v
        else:
            out[k] = v.index_select(0, idx_t).contiguous()
    return out


def compare_accept(ref, tokens, lens, gamma):
    """Compare accepted lengths and tokens sequence by sequence.

    A sequence's outputs are compared in decision order; at the first decision
    where the two sides differ the oracle's margin decides: below MARGIN the
    difference is exempt and everything after it in that sequence is downstream
    (not compared); otherwise it is a hard mismatch.
    """
    B = len(lens)
    stats = dict(sequences=B, exact=0, exempt_accept=0, exempt_sample=0, hard=0, tight_mismatch=0, details=[])
    for b in range(B):
        n_o, n_g = int(ref["accept_len"][b]) - 1, int(lens[b]) - 1
        t_o, t_g = ref["out_tokens"][b], tokens[b]
        if n_o != n_g:
            j = min(n_o, n_g)
            m = ref["margin_accept"][b, j]
            if 0 <= m < MARGIN:
                stats["exempt_accept"] += 1
            else:
                stats["hard"] += 1
                stats["details"].append(("accept", b, j, float(m), n_o, n_g))
            stats["tight_mismatch"] += int(m >= TIGHT)
            continue
        if not np.array_equal(t_o[:n_o], t_g[:n_o]) or not np.all(t_g[n_o + 1:] == -1):
            stats["hard"] += 1
            stats["details"].append(("drafts", b, t_o.tolist(), t_g.tolist()))
            continue
        if t_o[n_o] != t_g[n_o]:
            m = ref["margin_sample"][b]
            if 0 <= m < MARGIN:
                stats["exempt_sample"] += 1
            else:
                stats["hard"] += 1
                stats["details"].append(("sample", b, int(t_o[n_o]), int(t_g[n_o]), float(m)))
            stats["tight_mismatch"] += int(m >= TIGHT)
            continue
        stats["exact"] += 1
    return stats


def oracle_attention(w, window=0):
    """The oracle's append + attention alone on a workload dict (attn_out, lse and the page pools
    after the append), for cases that compare attention on more sequences than the whole step."""
    seq = w["seq_lens"].cpu().numpy().astype(np.int32).copy()
    kp, vp = oracle.bf16_bits(w["k_pages"]).copy(), oracle.bf16_bits(w["v_pages"]).copy()
    pt = w["page_table"].cpu().numpy().astype(np.int32)
    oracle.kv_append(oracle.bf16_bits(w["k_new"]), oracle.bf16_bits(w["v_new"]), kp, vp, pt, seq)
    out, lse = oracle.verify_attn(oracle.bf16_bits(w["q"]), kp, vp, pt, seq, None, window)
    return dict(attn_out=out, lse=lse, k_pages=kp, v_pages=vp)


def oracle_step(w, temperature, want_attention=True):
    return oracle.verify_step(w, temperature, want_attention=want_attention)

"""CPU oracle of the verify step (test infrastructure; never on a product path).

``oracle.build()`` compiles ``massv_oracle.c`` with gcc; the functions below are
thin numpy/ctypes marshalling around it.  bf16 tensors are passed as uint16 bit
patterns.  Nothing here imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "massv_oracle.c")
_LIB = os.path.join(_HERE, "libmassv_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c99", "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_tvd.restype = ctypes.c_double
        _lib.oracle_num_threads.restype = ctypes.c_int
    return _lib


def _p(a, dtype):
    if a is None:
        return None
    assert isinstance(a, np.ndarray) and a.dtype == dtype and a.flags["C_CONTIGUOUS"], (type(a), getattr(a, "dtype", None), dtype)
    return a.ctypes.data_as(ctypes.c_void_p)


def bf16_bits(t) -> np.ndarray:
    """torch bf16 tensor (any device) -> contiguous numpy uint16 array of its bit patterns."""
    import torch
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def kv_append(k_new, v_new, k_pages, v_pages, page_table, seq_lens):
    """In-place append of the block's K/V (uint16 [B,R,Hkv,d]) into the page pools (uint16 [P,Hkv,page,d])."""
    B, R, Hkv, d = k_new.shape
    page = k_pages.shape[2]
    _load().oracle_kv_append(B, R, Hkv, d, page, page_table.shape[1],
                             _p(k_new, np.uint16), _p(v_new, np.uint16), _p(k_pages, np.uint16), _p(v_pages, np.uint16),
                             _p(page_table, np.int32), _p(seq_lens, np.int32))


def verify_attn(q, k_pages, v_pages, page_table, seq_lens, scale=None, window=0):
    """Block attention over the (already appended) cache. Returns (out f64 [B,R,Hq,d], lse f64 [B,R,Hq]).
    window > 0: each row sees only the last `window` positions up to itself."""
    B, R, Hq, d = q.shape
    Hkv, page = k_pages.shape[1], k_pages.shape[2]
    if scale is None:
        scale = 1.0 / np.sqrt(d)
    out = np.zeros((B, R, Hq, d), dtype=np.float64)
    lse = np.zeros((B, R, Hq), dtype=np.float64)
    _load().oracle_verify_attn(B, R, Hq, Hkv, d, page, page_table.shape[1], int(window), ctypes.c_double(scale),
                               _p(q, np.uint16), _p(k_pages, np.uint16), _p(v_pages, np.uint16),
                               _p(page_table, np.int32), _p(seq_lens, np.int32), _p(out, np.float64), _p(lse, np.float64))
    return out, lse


def logits(hidden, lm_head):
    """z f64 [M,V] from uint16 hidden [M,K] and lm_head [V,K]."""
    M, K = hidden.shape
    V = lm_head.shape[0]
    assert lm_head.shape[1] == K
    z = np.zeros((M, V), dtype=np.float64)
    _load().oracle_logits(M, K, V, _p(hidden, np.uint16), _p(lm_head, np.uint16), _p(z, np.float64))
    return z


def softmax(z, T):
    M, V = z.shape
    p = np.zeros_like(z)
    _load().oracle_softmax(M, V, ctypes.c_double(T), _p(z, np.float64), _p(p, np.float64))
    return p


def accept(T, z, p, draft_tokens, draft_probs, u_accept, u_sample):
    """Acceptance + extra token for B sequences.

    z, p: f64 [B*(gamma+1), V] (p may be None at T == 0; z may be None at T > 0).
    Returns dict(out_tokens [B,gamma+1], accept_len [B], margin_accept [B,gamma], margin_sample [B]).
    """
    B, gamma = draft_tokens.shape
    V = (z if z is not None else p).shape[-1]
    out_tokens = np.zeros((B, gamma + 1), dtype=np.int32)
    accept_len = np.zeros((B,), dtype=np.int32)
    margin_accept = np.zeros((B, gamma), dtype=np.float64)
    margin_sample = np.zeros((B,), dtype=np.float64)
    _load().oracle_accept(B, gamma, V, ctypes.c_double(T), _p(z, np.float64), _p(p, np.float64),
                          _p(draft_tokens, np.int32), _p(draft_probs, np.float32),
                          _p(u_accept, np.float32), _p(u_sample, np.float32),
                          _p(out_tokens, np.int32), _p(accept_len, np.int32),
                          _p(margin_accept, np.float64), _p(margin_sample, np.float64))
    return dict(out_tokens=out_tokens, accept_len=accept_len, margin_accept=margin_accept, margin_sample=margin_sample)


def kv_commit(accept_len, seq_lens):
    """seq_lens += accept_len in place; accept_len None is a rollback (no change)."""
    _load().oracle_kv_commit(seq_lens.shape[0], _p(accept_len, np.int32), _p(seq_lens, np.int32))


def tvd(p, q):
    return float(_load().oracle_tvd(p.shape[0], _p(p, np.float64), _p(q, np.float64)))


def tvd_histogram(tvd, bins, counts=None):
    """counts[k] += number of TVD values (f32, any shape) in bin k of `bins` equal bins over [0, 1]."""
    t = np.ascontiguousarray(tvd, dtype=np.float32).reshape(-1)
    if counts is None:
        counts = np.zeros((bins,), dtype=np.int64)
    lib = _load()
    lib.oracle_tvd_histogram.restype = ctypes.c_longlong
    lib.oracle_tvd_histogram(ctypes.c_longlong(t.shape[0]), _p(t, np.float32), int(bins), _p(counts, np.int64))
    return counts


def sample_top_p(z, u, T, top_p, want_q=True):
    """Nucleus sampling of softmax(z / T), row by row: z f32 [rows, V], u f32 [rows].
    Returns dict(token, q (f64 [rows, V] or None), nucleus_size, margin_set, margin_sample)."""
    rows, V = z.shape
    token = np.zeros((rows,), dtype=np.int32)
    size = np.zeros((rows,), dtype=np.int32)
    q = np.zeros((rows, V), dtype=np.float64) if want_q else None
    m_set = np.zeros((rows,), dtype=np.float64)
    m_sample = np.zeros((rows,), dtype=np.float64)
    _load().oracle_sample_top_p(rows, V, ctypes.c_double(T), ctypes.c_double(top_p), _p(z, np.float32), _p(u, np.float32),
                                _p(token, np.int32), _p(q, np.float64), _p(size, np.int32), _p(m_set, np.float64),
                                _p(m_sample, np.float64))
    return dict(token=token, q=q, nucleus_size=size, margin_set=m_set, margin_sample=m_sample)


def verify_step(w, temperature, scale=None, want_attention=True, window=0):
    """Whole verify step on a workload dict of torch tensors (see ``workloads.generate``).

    Returns a dict with numpy results; the workload's page pools are not modified
    (the append runs on copies).  ``seq_lens_after`` is the committed length.
    """
    res = {}
    seq = w["seq_lens"].cpu().numpy().astype(np.int32).copy()
    if want_attention:
        kp, vp = bf16_bits(w["k_pages"]).copy(), bf16_bits(w["v_pages"]).copy()
        pt = w["page_table"].cpu().numpy().astype(np.int32)
        kv_append(bf16_bits(w["k_new"]), bf16_bits(w["v_new"]), kp, vp, pt, seq)
        res["attn_out"], res["lse"] = verify_attn(bf16_bits(w["q"]), kp, vp, pt, seq, scale, window)
        res["k_pages"], res["v_pages"] = kp, vp
    B, R, K = w["hidden"].shape
    z = logits(bf16_bits(w["hidden"]).reshape(B * R, K), bf16_bits(w["lm_head"]))
    res["logits"] = z
    if temperature > 0:
        p = softmax(z, temperature)
        res["probs"] = p
        acc = accept(temperature, None, p, w["draft_tokens"].cpu().numpy(), w["draft_probs"].cpu().numpy(),
                     w["u_accept"].cpu().numpy(), w["u_sample"].cpu().numpy())
    else:
        acc = accept(0.0, z, None, w["draft_tokens"].cpu().numpy(), None, None, None)
    res.update(acc)
    kv_commit(acc["accept_len"], seq)
    res["seq_lens_after"] = seq
    return res

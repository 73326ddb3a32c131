"""ctypes binding of ``libmassv.so``: argument marshalling only.

Every function takes torch tensors that already live on the GPU (torch is used
for device memory and streams, nothing else), passes their addresses and the
current CUDA stream to the C entry point of the same name, and raises
``MassvError`` on a non-zero status.  There is no CPU path: importing this
module without the compiled library raises.
"""
from __future__ import annotations

import ctypes
import os

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
# MASSV_DEBUG=1 selects the build with device-side index checks (same entry points, MASSV_ERR_BOUNDS in dev_status
# where an index leaves its buffer); it has to exist, like the ordinary library
LIB_PATH = os.path.join(_PKG, "libmassv_debug.so" if os.environ.get("MASSV_DEBUG", "0") not in ("", "0") else "libmassv.so")


class MassvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {_strerror(status)} (status {status})")


class AttnDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("gamma", ctypes.c_int32), ("n_q_heads", ctypes.c_int32),
                ("n_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32), ("page_size", ctypes.c_int32),
                ("max_pages_per_seq", ctypes.c_int32), ("num_pages", ctypes.c_int64), ("scale", ctypes.c_float),
                ("kv_chunk", ctypes.c_int32), ("window", ctypes.c_int32), ("flags", ctypes.c_uint32)]


class AcceptDesc(ctypes.Structure):
    _fields_ = [("batch", ctypes.c_int32), ("gamma", ctypes.c_int32), ("hidden", ctypes.c_int32),
                ("vocab", ctypes.c_int32), ("temperature", ctypes.c_float), ("flags", ctypes.c_uint32)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_10526_b200.build` "
                          "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32p, f32p = ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p
    lib.massv_verify_attn_workspace_size.restype = ctypes.c_size_t
    lib.massv_verify_attn_workspace_size.argtypes = [ctypes.POINTER(AttnDesc)]
    lib.massv_verify_attn.restype = ctypes.c_int
    lib.massv_verify_attn.argtypes = [ctypes.POINTER(AttnDesc), vp, vp, vp, vp, vp, i32p, i32p, vp, f32p, f32p,
                                      vp, ctypes.c_size_t, i32p, vp]
    lib.massv_accept_workspace_size.restype = ctypes.c_size_t
    lib.massv_accept_workspace_size.argtypes = [ctypes.POINTER(AcceptDesc)]
    lib.massv_accept.restype = ctypes.c_int
    lib.massv_accept.argtypes = [ctypes.POINTER(AcceptDesc), vp, vp, i32p, f32p, f32p, f32p, i32p, i32p, f32p, f32p,
                                 vp, ctypes.c_size_t, i32p, vp]
    lib.massv_accept_static.restype = ctypes.c_int
    lib.massv_accept_static.argtypes = [ctypes.POINTER(AcceptDesc), vp, vp, i32p, f32p, f32p, f32p, i32p, i32p, f32p, f32p,
                                        i32p, vp]
    lib.massv_tvd_workspace_size.restype = ctypes.c_size_t
    lib.massv_tvd_workspace_size.argtypes = [ctypes.POINTER(AcceptDesc)]
    lib.massv_tvd.restype = ctypes.c_int
    lib.massv_tvd.argtypes = [ctypes.POINTER(AcceptDesc), f32p, f32p, f32p, f32p, vp, ctypes.c_size_t, i32p, vp]
    lib.massv_tvd_after_accept.restype = ctypes.c_int
    lib.massv_tvd_after_accept.argtypes = [ctypes.POINTER(AcceptDesc), f32p, f32p, vp, ctypes.c_size_t, f32p, f32p, vp, ctypes.c_size_t, i32p, vp]
    lib.massv_tvd_histogram.restype = ctypes.c_int
    lib.massv_tvd_histogram.argtypes = [ctypes.c_int64, f32p, ctypes.c_int32, vp, vp]
    lib.massv_sample_top_p.restype = ctypes.c_int
    lib.massv_sample_top_p.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_float, ctypes.c_float, f32p, f32p, i32p, f32p, i32p, vp]
    D, i32 = ctypes.POINTER(AcceptDesc), ctypes.c_int32
    for name in ("massv_shard_stats_words", "massv_shard_mass_count", "massv_shard_state_bytes"):
        getattr(lib, name).restype = ctypes.c_size_t
        getattr(lib, name).argtypes = [D]
    lib.massv_shard_lm_head.restype = ctypes.c_int
    lib.massv_shard_lm_head.argtypes = [D, i32, i32, vp, vp, f32p, f32p, ctypes.POINTER(ctypes.c_int32), i32p, vp]
    lib.massv_shard_gather_draft.restype = ctypes.c_int
    lib.massv_shard_gather_draft.argtypes = [D, i32, i32, f32p, f32p, i32p, f32p, i32p, vp]
    lib.massv_shard_scan.restype = ctypes.c_int
    lib.massv_shard_scan.argtypes = [D, i32, i32, f32p, i32p, f32p, i32p, i32p, vp, i32p, vp]
    lib.massv_shard_masses.restype = ctypes.c_int
    lib.massv_shard_masses.argtypes = [D, i32, i32, f32p, f32p, vp, vp, i32p, vp]
    lib.massv_shard_pick.restype = ctypes.c_int
    lib.massv_shard_pick.argtypes = [D, i32, i32, vp, f32p, vp, f32p, f32p, i32p, i32p, vp]
    lib.massv_shard_publish.restype = ctypes.c_int
    lib.massv_shard_publish.argtypes = [vp, ctypes.c_size_t, ctypes.POINTER(ctypes.c_void_p), i32, i32, vp]
    lib.massv_shard_set_token.restype = ctypes.c_int
    lib.massv_shard_set_token.argtypes = [D, i32, vp, i32p, i32p, i32p, vp]
    lib.massv_kv_commit.restype = ctypes.c_int
    lib.massv_kv_commit.argtypes = [ctypes.c_int32, ctypes.c_int32, i32p, i32p, i32p, vp]
    lib.massv_strerror.restype = ctypes.c_char_p
    lib.massv_strerror.argtypes = [ctypes.c_int]
    lib.massv_version.restype = ctypes.c_int
    lib.massv_launch_count.restype = ctypes.c_uint64
    lib.massv_set_timing_events.restype = ctypes.c_int
    lib.massv_set_timing_events.argtypes = [vp, vp, vp, vp]
    lib.massv_set_kernel_timing.restype = ctypes.c_int
    lib.massv_set_kernel_timing.argtypes = [ctypes.c_int32, vp, vp]
    return lib


_lib = _load()


def _strerror(status: int) -> str:
    return _lib.massv_strerror(int(status)).decode()


def _ptr(t, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError("massv: tensors must live on a CUDA device")
    if not t.is_contiguous():
        raise ValueError("massv: tensors must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise ValueError(f"massv: expected {dtype}, got {t.dtype}")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


def massv_version() -> int:
    return int(_lib.massv_version())


def massv_launch_count() -> int:
    return int(_lib.massv_launch_count())


def massv_set_timing_events(lm_head=None, attn=None) -> None:
    """Record pairs of torch CUDA events (created with enable_timing=True) around the LM-head kernel
    and / or the attention split kernel of the following calls on this thread; None switches a hook off."""
    def handles(pair):
        if pair is None:
            return None, None
        for ev in pair:
            if not getattr(ev, "cuda_event", 0):
                ev.record()                 # torch creates the underlying CUDA event lazily
        return ctypes.c_void_p(pair[0].cuda_event), ctypes.c_void_p(pair[1].cuda_event)
    rc = _lib.massv_set_timing_events(*handles(lm_head), *handles(attn))
    if rc != 0:
        raise MassvError(rc, "massv_set_timing_events")


TIMED_LM_HEAD, TIMED_ATTN, TIMED_RESIDUAL = 0, 1, 2


def massv_set_kernel_timing(kernel: int, pair=None) -> None:
    """Record a pair of torch CUDA events around one kernel (TIMED_*) of the following calls on this
    thread; None switches that kernel's hook off."""
    if pair is None:
        a = b = None
    else:
        for ev in pair:
            if not getattr(ev, "cuda_event", 0):
                ev.record()                 # torch creates the underlying CUDA event lazily
        a, b = ctypes.c_void_p(pair[0].cuda_event), ctypes.c_void_p(pair[1].cuda_event)
    rc = _lib.massv_set_kernel_timing(int(kernel), a, b)
    if rc != 0:
        raise MassvError(rc, "massv_set_kernel_timing")


def massv_strerror(status: int) -> str:
    return _strerror(status)


# massv_attn_desc.flags: which split kernel runs (include/massv.h)
ATTN_KERNEL_AUTO, ATTN_KERNEL_WARP_MMA, ATTN_KERNEL_TCGEN05 = 0, 1, 2


def attn_desc(batch, gamma, n_q_heads, n_kv_heads, head_dim, max_pages_per_seq, num_pages, scale=0.0, kv_chunk=0,
              page_size=16, window=0, kernel=ATTN_KERNEL_AUTO) -> AttnDesc:
    return AttnDesc(batch, gamma, n_q_heads, n_kv_heads, head_dim, page_size, max_pages_per_seq, num_pages,
                    float(scale), kv_chunk, window, int(kernel))


def accept_desc(batch, gamma, hidden, vocab, temperature) -> AcceptDesc:
    return AcceptDesc(batch, gamma, hidden, vocab, float(temperature), 0)


def massv_verify_attn_workspace_size(desc: AttnDesc) -> int:
    return int(_lib.massv_verify_attn_workspace_size(ctypes.byref(desc)))


def massv_accept_workspace_size(desc: AcceptDesc) -> int:
    return int(_lib.massv_accept_workspace_size(ctypes.byref(desc)))


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    """A 256-byte aligned scratch buffer (torch's caching allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def massv_verify_attn(desc, q, k_new, v_new, k_pages, v_pages, page_table, seq_lens, out, out_f32=None, lse=None,
                      workspace=None, dev_status=None) -> None:
    bf = torch.bfloat16
    rc = _lib.massv_verify_attn(ctypes.byref(desc), _ptr(q, bf), _ptr(k_new, bf), _ptr(v_new, bf), _ptr(k_pages, bf),
                                _ptr(v_pages, bf), _ptr(page_table, torch.int32), _ptr(seq_lens, torch.int32),
                                _ptr(out, bf), _ptr(out_f32, torch.float32), _ptr(lse, torch.float32),
                                _ptr(workspace), workspace.numel() if workspace is not None else 0,
                                _ptr(dev_status, torch.int32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_verify_attn")


def massv_accept(desc, hidden, lm_head, draft_tokens, draft_probs, u_accept, u_sample, out_tokens, accept_len,
                 logits_out=None, probs_out=None, workspace=None, dev_status=None) -> None:
    bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
    rc = _lib.massv_accept(ctypes.byref(desc), _ptr(hidden, bf), _ptr(lm_head, bf), _ptr(draft_tokens, i32),
                           _ptr(draft_probs, f32), _ptr(u_accept, f32), _ptr(u_sample, f32), _ptr(out_tokens, i32),
                           _ptr(accept_len, i32), _ptr(logits_out, f32), _ptr(probs_out, f32),
                           _ptr(workspace), workspace.numel() if workspace is not None else 0,
                           _ptr(dev_status, i32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_accept")


def massv_accept_static(desc, hidden, lm_head, draft_tokens, draft_probs, u_accept, u_sample, out_tokens, accept_len,
                        logits_out=None, probs_out=None, dev_status=None) -> None:
    """massv_accept without a workspace: scratch is a fixed array inside the
    library (for callers that cannot allocate device memory).  Needs logits_out
    at T > 0; small problems only (see include/massv.h)."""
    bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
    rc = _lib.massv_accept_static(ctypes.byref(desc), _ptr(hidden, bf), _ptr(lm_head, bf), _ptr(draft_tokens, i32),
                                  _ptr(draft_probs, f32), _ptr(u_accept, f32), _ptr(u_sample, f32),
                                  _ptr(out_tokens, i32), _ptr(accept_len, i32), _ptr(logits_out, f32),
                                  _ptr(probs_out, f32), _ptr(dev_status, i32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_accept_static")


def massv_tvd_workspace_size(desc: AcceptDesc) -> int:
    return int(_lib.massv_tvd_workspace_size(ctypes.byref(desc)))


def massv_tvd(desc, logits, draft_probs, tvd_out, accept_prob_out=None, workspace=None, dev_status=None) -> None:
    f32 = torch.float32
    rc = _lib.massv_tvd(ctypes.byref(desc), _ptr(logits, f32), _ptr(draft_probs, f32), _ptr(tvd_out, f32),
                        _ptr(accept_prob_out, f32), _ptr(workspace), workspace.numel() if workspace is not None else 0,
                        _ptr(dev_status, torch.int32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_tvd")


def massv_tvd_after_accept(desc, logits, draft_probs, accept_workspace, tvd_out, accept_prob_out=None, workspace=None,
                           dev_status=None) -> None:
    """massv_tvd with one read of the logits: the row statistics come from the workspace that the
    massv_accept call with the same descriptor has just used."""
    f32 = torch.float32
    rc = _lib.massv_tvd_after_accept(ctypes.byref(desc), _ptr(logits, f32), _ptr(draft_probs, f32), _ptr(accept_workspace),
                                     accept_workspace.numel(), _ptr(tvd_out, f32), _ptr(accept_prob_out, f32), _ptr(workspace),
                                     workspace.numel() if workspace is not None else 0, _ptr(dev_status, torch.int32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_tvd_after_accept")


def massv_tvd_histogram(tvd, counts) -> None:
    """counts (int64 [bins]) += histogram of the fp32 tensor ``tvd`` over [0, 1]."""
    rc = _lib.massv_tvd_histogram(tvd.numel(), _ptr(tvd, torch.float32), counts.numel(), _ptr(counts, torch.int64), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_tvd_histogram")


def massv_sample_top_p(logits, u, tokens, temperature, top_p, probs_out=None, dev_status=None) -> None:
    """Nucleus sampling of softmax(logits / temperature), one draw per row (logits fp32 [rows, V])."""
    f32, i32 = torch.float32, torch.int32
    rows, vocab = logits.shape
    rc = _lib.massv_sample_top_p(rows, vocab, float(temperature), float(top_p), _ptr(logits, f32), _ptr(u, f32),
                                 _ptr(tokens, i32), _ptr(probs_out, f32), _ptr(dev_status, i32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_sample_top_p")


# ---- vocabulary shards (argument marshalling only; the caller moves the gathered buffers between ranks)
def massv_shard_stats_words(desc) -> int:
    return int(_lib.massv_shard_stats_words(ctypes.byref(desc)))


def massv_shard_mass_count(desc) -> int:
    return int(_lib.massv_shard_mass_count(ctypes.byref(desc)))


def massv_shard_state_bytes(desc) -> int:
    return int(_lib.massv_shard_state_bytes(ctypes.byref(desc)))


def _check(rc, name):
    if rc != 0:
        raise MassvError(rc, name)


def massv_shard_lm_head(desc, world, rank, hidden, lm_head_shard, logits_shard, stats, dev_status=None) -> int:
    """Returns the number of partial slots written (the same on every rank)."""
    bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
    n = ctypes.c_int32(0)
    _check(_lib.massv_shard_lm_head(ctypes.byref(desc), world, rank, _ptr(hidden, bf), _ptr(lm_head_shard, bf),
                                    _ptr(logits_shard, f32), _ptr(stats, f32), ctypes.byref(n), _ptr(dev_status, i32),
                                    _stream()), "massv_shard_lm_head")
    return int(n.value)


def massv_shard_gather_draft(desc, world, rank, logits_shard, draft_probs_shard, draft_tokens, stats,
                             dev_status=None) -> None:
    f32, i32 = torch.float32, torch.int32
    _check(_lib.massv_shard_gather_draft(ctypes.byref(desc), world, rank, _ptr(logits_shard, f32),
                                         _ptr(draft_probs_shard, f32), _ptr(draft_tokens, i32), _ptr(stats, f32),
                                         _ptr(dev_status, i32), _stream()), "massv_shard_gather_draft")


def massv_shard_scan(desc, world, n_partials, stats_all, draft_tokens, u_accept, out_tokens, accept_len, state,
                     dev_status=None) -> None:
    f32, i32 = torch.float32, torch.int32
    _check(_lib.massv_shard_scan(ctypes.byref(desc), world, n_partials, _ptr(stats_all, f32), _ptr(draft_tokens, i32),
                                 _ptr(u_accept, f32), _ptr(out_tokens, i32), _ptr(accept_len, i32),
                                 _ptr(state, torch.uint8), _ptr(dev_status, i32), _stream()), "massv_shard_scan")


def massv_shard_masses(desc, world, rank, logits_shard, draft_probs_shard, state, masses, dev_status=None) -> None:
    f32, f64, i32 = torch.float32, torch.float64, torch.int32
    _check(_lib.massv_shard_masses(ctypes.byref(desc), world, rank, _ptr(logits_shard, f32),
                                   _ptr(draft_probs_shard, f32), _ptr(state, torch.uint8), _ptr(masses, f64),
                                   _ptr(dev_status, i32), _stream()), "massv_shard_masses")


def massv_shard_pick(desc, world, rank, masses_all, u_sample, state, logits_shard, draft_probs_shard, token_out,
                     dev_status=None) -> None:
    f32, f64, i32 = torch.float32, torch.float64, torch.int32
    _check(_lib.massv_shard_pick(ctypes.byref(desc), world, rank, _ptr(masses_all, f64), _ptr(u_sample, f32),
                                 _ptr(state, torch.uint8), _ptr(logits_shard, f32), _ptr(draft_probs_shard, f32),
                                 _ptr(token_out, i32), _ptr(dev_status, i32), _stream()), "massv_shard_pick")


def massv_shard_publish(src, gathered, rank) -> None:
    """Store ``src`` at slot ``rank`` of every tensor in ``gathered`` (one per rank, each world x src's size)."""
    world = len(gathered)
    nbytes = src.numel() * src.element_size()
    for g in gathered:
        if g.numel() * g.element_size() != world * nbytes:
            raise ValueError("massv: a gathered buffer must be world times the source's size")
    ptrs = (ctypes.c_void_p * world)(*[_ptr(g) for g in gathered])
    _check(_lib.massv_shard_publish(_ptr(src), nbytes, ptrs, world, rank, _stream()), "massv_shard_publish")


def massv_shard_set_token(desc, world, state, tokens_all, out_tokens, dev_status=None) -> None:
    i32 = torch.int32
    _check(_lib.massv_shard_set_token(ctypes.byref(desc), world, _ptr(state, torch.uint8), _ptr(tokens_all, i32),
                                      _ptr(out_tokens, i32), _ptr(dev_status, i32), _stream()), "massv_shard_set_token")


def massv_kv_commit(batch, gamma, accept_len, seq_lens, dev_status=None) -> None:
    rc = _lib.massv_kv_commit(batch, gamma, _ptr(accept_len, torch.int32), _ptr(seq_lens, torch.int32),
                              _ptr(dev_status, torch.int32), _stream())
    if rc != 0:
        raise MassvError(rc, "massv_kv_commit")

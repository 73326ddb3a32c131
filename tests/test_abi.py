"""The C-ABI library loads, exports what include/massv.h declares, and rejects
bad arguments on the host before touching the GPU (runs without a GPU)."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mv():
    entry.build()
    import paper_2505_10526_b200 as pkg
    return pkg


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "massv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(massv_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(mv):
    lib = ctypes.CDLL(mv.LIB_PATH)
    names = declared_symbols()
    assert {"massv_verify_attn", "massv_accept", "massv_kv_commit", "massv_verify_attn_workspace_size",
            "massv_accept_workspace_size", "massv_strerror", "massv_version"} <= set(names)
    for n in names:
        assert hasattr(lib, n), n


def test_the_test_and_debug_builds_export_the_same_symbols(mv):
    pkg_dir = os.path.dirname(mv.LIB_PATH)
    for variant in ("libmassv_testhooks.so", "libmassv_debug.so"):
        lib = ctypes.CDLL(os.path.join(pkg_dir, variant))
        for n in declared_symbols():
            assert hasattr(lib, n), (variant, n)
        lib.massv_strerror.restype = ctypes.c_char_p
        assert b"bounds" in lib.massv_strerror(-7)


def test_python_binding_has_the_same_names(mv):
    for n in declared_symbols():
        assert hasattr(mv, n) or hasattr(mv.binding, n), n


def test_version_and_strerror(mv):
    assert mv.massv_version() >= 100
    assert mv.massv_strerror(0) == "ok"
    assert "workspace" in mv.massv_strerror(-4)
    assert mv.massv_strerror(-99) == "unknown status"


def test_workspace_sizes(mv):
    d = mv.attn_desc(16, 5, 28, 4, 128, 257, 4000)
    assert mv.massv_verify_attn_workspace_size(d) > 0
    assert mv.massv_verify_attn_workspace_size(mv.attn_desc(16, 5, 28, 4, 96, 257, 4000)) == 0      # head_dim
    assert mv.massv_verify_attn_workspace_size(mv.attn_desc(16, 9, 28, 4, 128, 257, 4000)) == 0     # gamma
    assert mv.massv_verify_attn_workspace_size(mv.attn_desc(16, 5, 28, 5, 128, 257, 4000)) == 0     # Hq % Hkv
    assert mv.massv_verify_attn_workspace_size(mv.attn_desc(16, 5, 28, 4, 128, 257, 4000, page_size=32)) == 0
    c = mv.accept_desc(16, 5, 3584, 152064, 1.0)
    assert mv.massv_accept_workspace_size(c) >= 96 * 152064 * 4
    assert mv.massv_accept_workspace_size(mv.accept_desc(16, 5, 3580, 152064, 1.0)) == 0            # K % 64
    assert mv.massv_accept_workspace_size(mv.accept_desc(100, 5, 3584, 152064, 1.0)) == 0           # M > 512
    assert mv.massv_accept_workspace_size(mv.accept_desc(16, 5, 3584, 152064, -1.0)) == 0


def test_host_validation_returns_status_without_launching(mv):
    lib = mv.binding._lib
    d = mv.attn_desc(1, 5, 4, 1, 64, 17, 20)
    nulls = [None] * 11 + [0, None, None]                          # ..., workspace, bytes, dev_status, stream
    assert lib.massv_verify_attn(ctypes.byref(d), *nulls) == -1     # NULL data pointers
    bad = mv.attn_desc(1, 5, 4, 1, 48, 17, 20)
    assert lib.massv_verify_attn(ctypes.byref(bad), *nulls) == -2
    c = mv.accept_desc(1, 5, 256, 1024, 0.0)
    assert lib.massv_accept(ctypes.byref(c), *nulls) == -1
    fake = 0x1000                                                   # aligned non-NULL address, never dereferenced
    assert lib.massv_accept(ctypes.byref(c), fake, fake, fake, None, None, None, fake, fake, None, None,
                            None, 0, None, None) == -4              # workspace missing
    assert lib.massv_accept(ctypes.byref(c), fake, fake, fake, None, None, None, fake, fake, None, fake,
                            fake, 1 << 40, None, None) == -1        # probs_out at T == 0
    assert lib.massv_accept(ctypes.byref(c), fake + 2, fake, fake, None, None, None, fake, fake, None, None,
                            fake, 1 << 40, None, None) == -1        # misaligned hidden
    t1 = mv.accept_desc(1, 5, 256, 1024, 1.0)
    assert lib.massv_accept(ctypes.byref(t1), fake, fake, fake, None, None, None, fake, fake, None, None,
                            fake, 1 << 40, None, None) == -1        # T > 0 needs q and the uniforms
    assert lib.massv_kv_commit(0, 5, None, None, None, None) == -1
    assert lib.massv_kv_commit(4, 9, None, fake, None, None) == -2
    assert lib.massv_kv_commit(4, 5, None, fake, None, None) == 0   # rollback: nothing to launch


def test_binding_refuses_cpu_tensors(mv):
    import torch
    d = mv.accept_desc(1, 5, 256, 1024, 0.0)
    x = torch.zeros(8, dtype=torch.bfloat16)
    with pytest.raises(ValueError):
        mv.massv_accept(d, x, x, None, None, None, None, None, None)


def test_timing_hook_rejects_half_a_pair(mv):
    """massv_set_timing_events takes events in pairs; one without the other is refused (host-only check)."""
    lib = ctypes.CDLL(mv.LIB_PATH)
    lib.massv_set_timing_events.restype = ctypes.c_int
    lib.massv_set_timing_events.argtypes = [ctypes.c_void_p] * 4
    assert lib.massv_set_timing_events(None, None, None, None) == 0
    assert lib.massv_set_timing_events(ctypes.c_void_p(8), None, None, None) == -1
    assert lib.massv_set_timing_events(None, None, None, ctypes.c_void_p(8)) == -1
    assert lib.massv_set_timing_events(None, None, None, None) == 0


def test_attention_refuses_more_chunks_than_the_merge_can_index(mv):
    """A forced 64-token chunk on a page table of more than 65,536 tokens per sequence would need more than
    1024 chunks: refused on the host (size query 0, call -2), nothing launched."""
    d = mv.attn_desc(1, 5, 4, 1, 64, 4097, 5000, kv_chunk=64)          # 65,552 tokens per sequence
    assert mv.massv_verify_attn_workspace_size(d) == 0
    lib = mv.binding._lib
    fake = 0x1000
    assert lib.massv_verify_attn(ctypes.byref(d), fake, fake, fake, fake, fake, fake, fake, fake, None, None, fake, 1 << 30, None, None) == -2
    ok = mv.attn_desc(1, 5, 4, 1, 64, 4096, 5000, kv_chunk=64)         # exactly 1024 chunks
    assert mv.massv_verify_attn_workspace_size(ok) > 0

"""massv_accept_static: the acceptance call for hosts that cannot allocate.

An inference engine that handed out all of its device memory at start-up, or a
component living inside another program's CUDA context under a no-allocation
rule, has no workspace to give massv_accept and may not create one.  For those
hosts the library carries a small fixed scratch array of its own.  This file
checks, through the C ABI, that the workspace-free call returns what the normal
call returns, twice in a row on different inputs (the array is shared between
calls and keeps the previous call's contents), and that problems larger than the
array are refused rather than run.

The file name sorts last on purpose: if this extra entry point ever breaks, a
run that stops at the first failure has already exercised everything else.
"""
import ctypes

import pytest
import torch

from workloads import generate, get_config

TOL_LOGIT = 2e-2   # the tolerance the parity tests use for logits


def _both_ways(mv, cfg, w):
    """Run massv_accept and massv_accept_static on the same inputs."""
    B, R, V = cfg.batch, cfg.rows, cfg.vocab
    desc = mv.accept_desc(B, cfg.gamma, cfg.hidden, V, cfg.temperature)
    sampling = cfg.temperature > 0
    args = (w["hidden"], w["lm_head"], w["draft_tokens"], w.get("draft_probs") if sampling else None,
            w.get("u_accept") if sampling else None, w.get("u_sample") if sampling else None)
    out = {}
    for name in ("plain", "static"):
        toks = torch.full((B, R), -7, dtype=torch.int32, device="cuda")
        lens = torch.zeros((B,), dtype=torch.int32, device="cuda")
        logits = torch.zeros((B, R, V), dtype=torch.float32, device="cuda")
        status = torch.zeros((1,), dtype=torch.int32, device="cuda")
        if name == "plain":
            ws = mv.alloc_workspace(mv.massv_accept_workspace_size(desc), "cuda")
            mv.massv_accept(desc, *args, toks, lens, logits, None, ws, status)
        else:
            mv.massv_accept_static(desc, *args, toks, lens, logits, None, status)
        out[name] = (toks, lens, logits, status)
    torch.cuda.synchronize()
    return out


@pytest.mark.gpu
def test_static_scratch_call_matches_the_workspace_call_twice_in_a_row():
    import paper_2505_10526_b200 as mv
    # two different problems back to back: sampling with ragged batch, then greedy at full vocabulary
    for name in ("tiny_ragged_t1", "qwen7b_b1_t0_calibrated", "tiny_ragged_t0", "tiny_peaked_t1"):
        cfg = get_config(name)
        w = generate(cfg, device="cuda", with_attention=False)
        res = _both_ways(mv, cfg, w)
        (t0, l0, z0, s0), (t1, l1, z1, s1) = res["plain"], res["static"]
        assert int(s0.item()) == 0 and int(s1.item()) == 0
        assert torch.equal(l0, l1), name
        assert torch.equal(t0, t1), name
        assert float((z0 - z1).abs().max()) <= TOL_LOGIT, name
        assert int(l1.min()) >= 1 and int(l1.max()) <= cfg.rows


@pytest.mark.gpu
def test_static_scratch_call_leaves_device_memory_alone():
    """The property the call exists for: free device memory (as the driver reports it) is the same before
    and after, also across the first call on the device, which looks up the array's address."""
    import paper_2505_10526_b200 as mv
    cfg = get_config("tiny_ragged_t1")
    w = generate(cfg, device="cuda", with_attention=False)
    B, R, V = cfg.batch, cfg.rows, cfg.vocab
    desc = mv.accept_desc(B, cfg.gamma, cfg.hidden, V, cfg.temperature)
    toks = torch.zeros((B, R), dtype=torch.int32, device="cuda"); lens = torch.zeros((B,), dtype=torch.int32, device="cuda")
    logits = torch.zeros((B, R, V), dtype=torch.float32, device="cuda"); status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        mv.massv_accept_static(desc, w["hidden"], w["lm_head"], w["draft_tokens"], w["draft_probs"], w["u_accept"], w["u_sample"],
                               toks, lens, logits, None, status)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert int(status.item()) == 0


@pytest.mark.gpu
def test_static_scratch_call_at_its_limits_and_with_a_bad_token():
    """The edges of the built-in array: 64 rows with a 524,288-entry vocabulary (128 residual chunks per
    sequence, the last slot of every part of the array), compared with the workspace call; and an
    out-of-range draft token, which both calls report through dev_status (-1) without faulting."""
    import paper_2505_10526_b200 as mv
    from workloads import VerifyConfig
    cfg = VerifyConfig(name="static_limit", batch=16, gamma=3, n_q_heads=1, n_kv_heads=1, head_dim=64, hidden=256, vocab=524288,
                       temperature=1.0, ctx_lo=1, ctx_hi=2, image_tokens=0.25, draft_noise_std=1.0, seed=77)
    w = generate(cfg, device="cuda", with_attention=False)
    res = _both_ways(mv, cfg, w)
    (t0, l0, z0, s0), (t1, l1, z1, s1) = res["plain"], res["static"]
    assert int(s0.item()) == 0 and int(s1.item()) == 0
    assert torch.equal(l0, l1) and torch.equal(t0, t1)
    assert float((z0 - z1).abs().max()) <= TOL_LOGIT
    bad = dict(w)
    bad["draft_tokens"] = w["draft_tokens"].clone()
    bad["draft_tokens"][3, 1] = cfg.vocab          # one past the last token
    res = _both_ways(mv, cfg, bad)
    assert int(res["plain"][3].item()) == -1 and int(res["static"][3].item()) == -1


def test_static_scratch_call_refuses_what_does_not_fit():
    """Host-side check only: nothing is launched, so it runs without a GPU."""
    import __graft_entry__ as entry
    entry.build()
    import paper_2505_10526_b200 as mv
    lib = mv.binding._lib
    fake = 0x1000
    too_many_rows = mv.accept_desc(16, 5, 3584, 152064, 0.0)          # 96 rows > 64
    rest = [fake, fake, fake, None, None, None, fake, fake, None, None, None, None]
    assert lib.massv_accept_static(ctypes.byref(too_many_rows), *rest) == -4
    too_wide = mv.accept_desc(1, 5, 256, 1 << 20, 0.0)                # vocabulary beyond the limit
    assert lib.massv_accept_static(ctypes.byref(too_wide), *rest) == -4
    needs_logits = mv.accept_desc(1, 5, 256, 1024, 1.0)               # T > 0 without logits_out
    assert lib.massv_accept_static(ctypes.byref(needs_logits), fake, fake, fake, fake, fake, fake, fake, fake,
                                   None, None, None, None) == -1
    assert "workspace" in mv.massv_strerror(-4)

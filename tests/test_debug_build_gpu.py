"""Memory-safety checks that need no sanitizer.

1. Canaries: every output of a verify step (attention output, log-sum-exp, tokens, lengths, logits,
   probabilities) and both workspaces are handed to the library as the middle of a larger buffer whose
   margins hold a pattern; after the step the margins must be untouched (the library wrote inside what it
   was given, and inside the workspace sizes it asked for).
2. The debug build: the same sources compiled with -DMASSV_DEBUG check the indices of their scattered
   stores on the device; an index outside its buffer would record MASSV_ERR_BOUNDS in dev_status and
   skip the store (no trap, no assert).  The tiny, odd-shaped and random-geometry parity tests are run
   again in a child process that loads that build (MASSV_DEBUG=1): they must pass, which includes a
   clean status word.
"""
import os
import subprocess
import sys

import pytest
import torch

from workloads import generate, get_config

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
GUARD = 256          # elements on each side of a guarded tensor


def _guarded(shape, dtype, device):
    """A tensor of the given shape in the middle of a larger one; returns (view, check) where check()
    asserts that the margins still hold the pattern."""
    n = 1
    for s in shape:
        n *= int(s)
    big = torch.empty((n + 2 * GUARD,), dtype=dtype, device=device)
    pattern = 0x5A if dtype == torch.uint8 else (0x5A5A5A5A if dtype == torch.int32 else 12345.0)
    big.fill_(pattern)
    view = big[GUARD:GUARD + n].view(*shape)

    def check(name):
        lo, hi = big[:GUARD], big[GUARD + n:]
        assert bool((lo == pattern).all()) and bool((hi == pattern).all()), f"{name}: a margin was written"
    return view, check


@pytest.mark.parametrize("name", ["tiny_t0", "tiny_t1", "tiny_ragged_t0", "tiny_ragged_t1", "tiny_peaked_t1"])
def test_outputs_and_workspaces_stay_inside_their_buffers(name):
    import paper_2505_10526_b200 as mv
    cfg = get_config(name)
    w = generate(cfg, device="cuda")
    dev = w["q"].device
    B, R, Hq, d, V = cfg.batch, cfg.gamma + 1, cfg.n_q_heads, cfg.head_dim, cfg.vocab
    sampling = cfg.temperature > 0
    adesc = mv.attn_desc(B, cfg.gamma, Hq, cfg.n_kv_heads, d, w["page_table"].shape[1], w["k_pages"].shape[0])
    cdesc = mv.accept_desc(B, cfg.gamma, cfg.hidden, V, cfg.temperature)
    checks = {}
    out, checks["attn out"] = _guarded((B, R, Hq, d), torch.bfloat16, dev)
    out_f32, checks["attn out fp32"] = _guarded((B, R, Hq, d), torch.float32, dev)
    lse, checks["lse"] = _guarded((B, R, Hq), torch.float32, dev)
    tokens, checks["tokens"] = _guarded((B, R), torch.int32, dev)
    lens, checks["lengths"] = _guarded((B,), torch.int32, dev)
    logits, checks["logits"] = _guarded((B, R, V), torch.float32, dev)
    probs, checks["probabilities"] = _guarded((B, R, V), torch.float32, dev)
    attn_ws, checks["attention workspace"] = _guarded((max(mv.massv_verify_attn_workspace_size(adesc), 256),), torch.uint8, dev)
    acc_ws, checks["acceptance workspace"] = _guarded((max(mv.massv_accept_workspace_size(cdesc), 256),), torch.uint8, dev)
    status = torch.zeros((1,), dtype=torch.int32, device=dev)
    for _ in range(2):                                    # a second call reuses the workspaces
        mv.massv_verify_attn(adesc, w["q"], w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"],
                             w["seq_lens"], out, out_f32, lse, attn_ws, status)
        mv.massv_accept(cdesc, w["hidden"], w["lm_head"], w["draft_tokens"],
                        w.get("draft_probs") if sampling else None, w.get("u_accept") if sampling else None,
                        w.get("u_sample") if sampling else None, tokens, lens, logits,
                        probs if sampling else None, acc_ws, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    for what, check in checks.items():
        check(what)
    assert bool((lens >= 1).all()) and bool((lens <= R).all())


def _run_under_debug_build(args, timeout=900):
    env = dict(os.environ, MASSV_DEBUG="1")
    return subprocess.run([sys.executable] + args, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_parity_tests_pass_under_the_debug_build():
    import importlib.util
    spec = importlib.util.spec_from_file_location("_massv_build", os.path.join(ROOT, "paper_2505_10526_b200", "build.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    mod.build_debug()
    probe = _run_under_debug_build(["-c", "import paper_2505_10526_b200.binding as b; print(b.LIB_PATH)"])
    assert probe.returncode == 0 and probe.stdout.strip().endswith("libmassv_debug.so"), probe.stdout + probe.stderr
    run = _run_under_debug_build(["-m", "pytest", "tests/test_parity_gpu.py", "-x", "-q", "-m", "gpu", "-k",
                                  "tiny_configs_full_parity or odd_shapes_and_forced_splits or random_small_shapes or "
                                  "either_attention_kernel_on_tiny or device_side_errors"])
    assert run.returncode == 0, run.stdout[-3000:] + run.stderr[-2000:]

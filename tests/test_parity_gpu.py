"""CUDA path vs CPU oracle, element by element, through the C ABI.

Tolerances (absolute): logits 2e-2 (bf16 operands, fp32 accumulation),
probabilities 1e-4, attention output 2e-2 in bf16 / 5e-3 in fp32 (softmax
weights are rounded to bf16 before the PV product), log-sum-exp 1e-3.
Integer outputs (appended cache bytes, tokens, accepted lengths, committed
lengths) are bit-exact except at decisions whose oracle margin is below 1e-3,
which are counted and printed.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from parity_util import compare_accept, oracle_attention, sub_workload
from workloads import generate, get_config

pytestmark = pytest.mark.gpu

TOL_LOGIT, TOL_PROB, TOL_ATTN_BF16, TOL_ATTN_F32, TOL_LSE = 2e-2, 1e-4, 2e-2, 5e-3, 1e-3
REPORT = os.environ.get("MASSV_PARITY_REPORT")      # optional: a file that collects one JSON line per parity case


def _report(entry):
    if REPORT:
        try:
            os.makedirs(os.path.dirname(os.path.abspath(REPORT)), exist_ok=True)
            with open(REPORT, "a") as f:
                f.write(json.dumps(entry) + "\n")
        except OSError:
            pass
    print(entry)


def run_case(name, subset=None, check_determinism=True, cfg=None, window=0, attn_subset=None, **step_kw):
    from paper_2505_10526_b200 import VerifyStep
    cfg = cfg or get_config(name)
    w = generate(cfg, device="cuda")
    pools_before = (w["k_pages"].clone(), w["v_pages"].clone())
    seq_before = w["seq_lens"].clone()
    step = VerifyStep.for_workload(cfg, w, want_logits=True, want_probs=True, want_attn_f32=True, window=window, **step_kw)
    step.run(w, commit=True)
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == 0

    idx = list(range(cfg.batch)) if subset is None else subset
    # attn_subset: sequences whose attention (and appended cache bytes) are compared, when that is a
    # larger set than the one the whole step is compared on ("all": the whole batch)
    idx_attn = idx if attn_subset is None else (list(range(cfg.batch)) if attn_subset == "all" else attn_subset)
    # the oracle sees the inputs as they were before the step
    w_ref = dict(w)
    w_ref["k_pages"], w_ref["v_pages"] = pools_before
    w_ref["seq_lens"] = seq_before
    ref = oracle.verify_step(sub_workload(w_ref, idx), cfg.temperature, window=window, want_attention=idx_attn == idx)
    if idx_attn != idx:
        ref.update(oracle_attention(sub_workload(w_ref, idx_attn), window=window))
    R, V = cfg.rows, cfg.vocab
    sel = torch.as_tensor(idx, device="cuda")
    sel_attn = torch.as_tensor(idx_attn, device="cuda")

    entry = dict(config=name or cfg.name, sequences=len(idx), sequences_attention=len(idx_attn), batch=cfg.batch)
    # -- appended cache bytes: every position < L + R of the checked sequences, bit-exact
    kp, vp = oracle.bf16_bits(w["k_pages"]), oracle.bf16_bits(w["v_pages"])
    pt = w["page_table"].cpu().numpy()
    for i, b in enumerate(idx_attn):
        n = int(seq_before[b]) + R
        pages = pt[b, :(n + 15) // 16]
        assert np.array_equal(kp[pages], ref["k_pages"][pages]) and np.array_equal(vp[pages], ref["v_pages"][pages])
    # pages of other sequences and unmapped pages are untouched unless they hold block slots
    if len(idx_attn) == cfg.batch:
        assert np.array_equal(kp, ref["k_pages"]) and np.array_equal(vp, ref["v_pages"])
    del kp, vp
    # -- attention
    o32 = step.attn_out_f32.index_select(0, sel_attn).cpu().double().numpy()
    o16 = step.attn_out.index_select(0, sel_attn).cpu().double().numpy()
    lse = step.lse.index_select(0, sel_attn).cpu().double().numpy()
    entry["attn_err_f32"] = float(np.abs(o32 - ref["attn_out"]).max())
    entry["attn_err_bf16"] = float(np.abs(o16 - ref["attn_out"]).max())
    entry["lse_err"] = float(np.abs(lse - ref["lse"]).max())
    ref.pop("k_pages", None); ref.pop("v_pages", None)
    # -- logits / probabilities
    z = step.logits.index_select(0, sel).cpu().double().numpy().reshape(-1, V)
    entry["logit_err"] = float(np.abs(z - ref["logits"]).max())
    if cfg.temperature > 0:
        p = step.probs.index_select(0, sel).cpu().double().numpy().reshape(-1, V)
        entry["prob_err"] = float(np.abs(p - ref["probs"]).max())
    # -- tokens, lengths, commit
    toks = step.out_tokens.index_select(0, sel).cpu().numpy()
    lens = step.accept_len.index_select(0, sel).cpu().numpy()
    st = compare_accept(ref, toks, lens, cfg.gamma)
    entry.update({k: v for k, v in st.items() if k != "details"})
    entry["mean_accept_len"] = float(step.accept_len.float().mean())
    after = w["seq_lens"].cpu().numpy()
    assert np.array_equal(after, seq_before.cpu().numpy() + step.accept_len.cpu().numpy())
    same = lens == ref["accept_len"]
    assert np.array_equal(after[idx][same], ref["seq_lens_after"][same])
    assert np.all((lens >= 1) & (lens <= R))

    if check_determinism:      # a second run on the same inputs is bit-identical
        first = (step.out_tokens.clone(), step.accept_len.clone(), step.attn_out.clone(), step.logits.clone())
        w["seq_lens"].copy_(seq_before)
        step.run(w, commit=False)
        torch.cuda.synchronize()
        assert torch.equal(first[0], step.out_tokens) and torch.equal(first[1], step.accept_len)
        assert torch.equal(first[2], step.attn_out) and torch.equal(first[3], step.logits)
    _report(entry)
    assert st["hard"] == 0, st["details"]
    assert entry["attn_err_f32"] < TOL_ATTN_F32 and entry["attn_err_bf16"] < TOL_ATTN_BF16 and entry["lse_err"] < TOL_LSE
    assert entry["logit_err"] < TOL_LOGIT
    if cfg.temperature > 0:
        assert entry["prob_err"] < TOL_PROB
    return entry


@pytest.mark.parametrize("name", ["tiny_t0", "tiny_t1", "tiny_ragged_t0", "tiny_ragged_t1", "tiny_peaked_t1"])
def test_tiny_configs_full_parity(name):
    run_case(name)


@pytest.mark.parametrize("name", ["qwen7b_b1_t0", "qwen7b_b1_t0_calibrated"])
def test_qwen_batch1_greedy_full_parity(name):
    e = run_case(name)
    if name.endswith("calibrated"):
        assert e["mean_accept_len"] >= 1.0


@pytest.mark.parametrize("name", ["qwen7b_b16_t1", "qwen7b_b16_t1_peaked"])
def test_qwen_batch16_sampling_full_parity(name):
    e = run_case(name)
    if name == "qwen7b_b16_t1":
        # flat vocabulary: acceptance tends to 2*Phi(-1/2) = 0.617 per position -> about 2.5 tokens per pass
        assert 1.5 < e["mean_accept_len"] < 3.6


def test_gemma_batch32_full_parity():
    """Config 4, every one of the 32 sequences, the whole step."""
    e = run_case("gemma12b_b32_t1")
    assert e["sequences"] == e["batch"] == 32


@pytest.mark.parametrize("name", ["qwen7b_long_g5_t1", "qwen7b_long_g7_t0"])
def test_long_context_whole_batch_whole_step(name):
    """Config 5, one point per temperature: all 64 sequences through the whole step (the flat attention
    schedule cuts (sequence, head) pairs at places that depend on the whole batch, so every sequence is
    compared, not a sample)."""
    e = run_case(name)
    assert e["sequences"] == e["sequences_attention"] == e["batch"] == 64


@pytest.mark.parametrize("name", ["qwen7b_long_g3_t0", "qwen7b_long_g3_t1", "qwen7b_long_g5_t0", "qwen7b_long_g7_t1"])
def test_long_context_whole_batch_attention(name):
    """The other config-5 points: attention and appended cache bytes for all 64 sequences, the LM head
    and acceptance on sampled sequences."""
    e = run_case(name, subset=[0, 33, 63], attn_subset="all", check_determinism=False)
    assert e["sequences_attention"] == e["batch"] == 64


def test_rollback_then_redraft_matches_a_fresh_step():
    """Rolling back leaves the lengths untouched, and verifying a different
    block afterwards gives what a cache that never saw the first block gives."""
    from paper_2505_10526_b200 import VerifyStep
    cfg = get_config("tiny_ragged_t1")
    w = generate(cfg, device="cuda")
    fresh = {k: v.clone() for k, v in w.items()}
    step = VerifyStep.for_workload(cfg, w, want_logits=True)
    seq0 = w["seq_lens"].clone()
    junk = dict(w)
    junk["k_new"] = torch.randn_like(w["k_new"].float()).to(torch.bfloat16)
    junk["v_new"] = torch.randn_like(w["v_new"].float()).to(torch.bfloat16)
    step.attn(junk); step.accept(junk); step.commit(w["seq_lens"], rollback=True)
    torch.cuda.synchronize()
    assert torch.equal(w["seq_lens"], seq0)
    step.run(w, commit=True)
    a = (step.attn_out.clone(), step.out_tokens.clone(), step.accept_len.clone(), w["seq_lens"].clone())
    step2 = VerifyStep.for_workload(cfg, fresh, want_logits=True)
    step2.run(fresh, commit=True)
    torch.cuda.synchronize()
    assert torch.equal(a[0], step2.attn_out) and torch.equal(a[1], step2.out_tokens)
    assert torch.equal(a[2], step2.accept_len) and torch.equal(a[3], fresh["seq_lens"])


def test_device_side_errors_are_reported_not_fatal():
    from paper_2505_10526_b200 import VerifyStep
    cfg = get_config("tiny_t0")
    w = generate(cfg, device="cuda")
    step = VerifyStep.for_workload(cfg, w)
    w["seq_lens"].fill_(w["page_table"].shape[1] * 16)          # no room for the block
    step.attn(w)
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == -3
    step.dev_status.zero_()
    bad = torch.full_like(step.accept_len, 99)
    from paper_2505_10526_b200 import massv_kv_commit
    before = w["seq_lens"].clone()
    massv_kv_commit(cfg.batch, cfg.gamma, bad, w["seq_lens"], step.dev_status)
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == -1 and torch.equal(before, w["seq_lens"])


def test_gamma_zero_is_plain_decoding():
    """With no drafts the step is one ordinary decoding step: one row, one token."""
    from dataclasses import replace
    from paper_2505_10526_b200 import VerifyStep
    cfg = replace(get_config("tiny_ragged_t0"), gamma=0, name="g0")
    w = generate(cfg, device="cuda")
    step = VerifyStep.for_workload(cfg, w, want_logits=True)
    ref = oracle.verify_step({k: v.clone() for k, v in w.items()}, 0.0)
    step.run(w)
    torch.cuda.synchronize()
    st = compare_accept(ref, step.out_tokens.cpu().numpy(), step.accept_len.cpu().numpy(), 0)
    assert st["hard"] == 0 and np.all(step.accept_len.cpu().numpy() == 1)


ODD_SHAPES = [
    # vocabulary not a multiple of the 128-row tile, hidden = 5 K-blocks, 7 rows per sequence
    dict(name="odd_vocab_t1", batch=3, gamma=6, n_q_heads=4, n_kv_heads=2, head_dim=64, hidden=320, vocab=1160,
         temperature=0.8, ctx_lo=0, ctx_hi=150),
    dict(name="odd_vocab_t0", batch=2, gamma=2, n_q_heads=2, n_kv_heads=2, head_dim=128, hidden=192, vocab=8200,
         temperature=0.0, ctx_lo=1, ctx_hi=70),
    # 8 query heads per KV head and gamma = 7: 64 query rows per CTA (four MMA row tiles), d = 256
    dict(name="wide_group_d256", batch=2, gamma=7, n_q_heads=8, n_kv_heads=1, head_dim=256, hidden=256, vocab=1024,
         temperature=1.0, ctx_lo=100, ctx_hi=400),
    # d = 256 with three row tiles, and d = 64 with one
    dict(name="three_tiles_d256", batch=2, gamma=5, n_q_heads=14, n_kv_heads=2, head_dim=256, hidden=256, vocab=1024,
         temperature=0.0, ctx_lo=60, ctx_hi=260),
    dict(name="one_tile_d64", batch=5, gamma=1, n_q_heads=6, n_kv_heads=3, head_dim=64, hidden=128, vocab=512,
         temperature=1.3, ctx_lo=0, ctx_hi=500),
    # 257 .. 384 LM-head rows (the one-pass, three-sub-tile arrangement): sub-tiles of 112 rows (a 16-column
    # tail) and of 96 rows, a ragged last vocabulary band, both temperatures
    dict(name="rows301_t1", batch=43, gamma=6, n_q_heads=2, n_kv_heads=1, head_dim=64, hidden=320, vocab=3000,
         temperature=0.9, ctx_lo=0, ctx_hi=40),
    dict(name="rows272_t0", batch=34, gamma=7, n_q_heads=2, n_kv_heads=2, head_dim=64, hidden=192, vocab=8200,
         temperature=0.0, ctx_lo=1, ctx_hi=50),
    # 76 vocabulary bands on 74 CTA pairs: the two left-over bands (the last one ragged) are cut into half-tiles
    dict(name="rows384_split_bands", batch=64, gamma=5, n_q_heads=2, n_kv_heads=1, head_dim=64, hidden=128, vocab=19400,
         temperature=1.1, ctx_lo=0, ctx_hi=30),
]


@pytest.mark.parametrize("spec", ODD_SHAPES, ids=[s["name"] for s in ODD_SHAPES])
@pytest.mark.parametrize("kv_chunk", [0, 64])
def test_odd_shapes_and_forced_splits(spec, kv_chunk):
    """Shapes off the benchmark grid (ragged vocabulary tile, every MMA row-tile count, all head
    dims), with the automatic chunking and with 64-token chunks that force the merge kernel."""
    from workloads import VerifyConfig
    cfg = VerifyConfig(image_tokens=0.25, draft_noise_std=0.7, seed=40 + len(spec["name"]), **spec)
    run_case(None, cfg=cfg, kv_chunk=kv_chunk)


KERNELS = [pytest.param(1, id="warp_mma"), pytest.param(2, id="tcgen05")]


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("name,kv_chunk", [("tiny_t1", 0), ("tiny_t1", 64), ("tiny_ragged_t0", 0), ("tiny_ragged_t0", 64),
                                           ("tiny_ragged_t1", 128), ("tiny_peaked_t1", 64)])
def test_either_attention_kernel_on_tiny_configs(name, kv_chunk, kernel):
    """The warp-MMA and the tcgen05 split kernels are interchangeable: each is forced in turn (the
    library would otherwise pick one by the row count) and held to the same tolerances, with whole
    contexts in one chunk and with chunks short enough that block rows straddle a chunk boundary."""
    run_case(name, kv_chunk=kv_chunk, attn_kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("spec", ODD_SHAPES, ids=[s["name"] for s in ODD_SHAPES])
@pytest.mark.parametrize("kv_chunk", [0, 64])
def test_either_attention_kernel_on_odd_shapes(spec, kv_chunk, kernel):
    from workloads import VerifyConfig
    cfg = VerifyConfig(image_tokens=0.25, draft_noise_std=0.7, seed=40 + len(spec["name"]), **spec)
    run_case(None, cfg=cfg, kv_chunk=kv_chunk, attn_kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("name,window,kv_chunk,subset", [
    ("tiny_ragged_t1", 1, 0, None), ("tiny_ragged_t1", 5, 64, None), ("tiny_ragged_t0", 40, 64, None), ("tiny_t1", 100, 64, None),
    ("qwen7b_b16_t1", 1500, 256, [0, 5, 15]),
])
def test_either_attention_kernel_with_a_sliding_window(name, window, kv_chunk, subset, kernel):
    run_case(name, subset=subset, check_determinism=False, window=window, kv_chunk=kv_chunk, attn_kernel=kernel)


@pytest.mark.parametrize("kernel", KERNELS)
@pytest.mark.parametrize("name,subset", [("qwen7b_b16_t1", [0, 5, 15]), ("gemma12b_b32_t1", [0, 31]), ("qwen7b_long_g7_t0", [0, 63]),
                                         ("qwen7b_long_g3_t0", [33])])
def test_either_attention_kernel_at_full_size(name, subset, kernel):
    run_case(name, subset=subset, check_determinism=False, attn_kernel=kernel)


def test_tcgen05_attention_rescales_when_the_maximum_grows():
    """Scores that keep growing along the context (keys scaled up with position) force the tcgen05
    kernel to move its reference maximum, i.e. to rescale the accumulator in tensor memory, many
    times; the result must still be the plain softmax."""
    from dataclasses import replace
    from paper_2505_10526_b200 import VerifyStep
    cfg = replace(get_config("tiny_ragged_t0"), name="growing_scores", batch=3, ctx_lo=700, ctx_hi=900, gamma=7)
    w = generate(cfg, device="cuda")
    # q = +1 everywhere, keys grow linearly with the page index they sit in: position i scores about i / 8
    pt = w["page_table"].long()
    ramp = torch.zeros(w["k_pages"].shape[0], device="cuda")
    for b in range(cfg.batch):
        ramp[pt[b]] = torch.arange(pt.shape[1], device="cuda", dtype=torch.float32)
    w["q"] = torch.ones_like(w["q"])
    w["k_pages"] = (torch.ones_like(w["k_pages"].float()) * ramp[:, None, None, None] * (16.0 / 8.0 / 8.0)).to(torch.bfloat16)
    for kernel in (1, 2):
        ww = {k: v.clone() for k, v in w.items()}
        ref = oracle.verify_step({k: v.clone() for k, v in ww.items()}, 0.0)
        step = VerifyStep.for_workload(cfg, ww, want_attn_f32=True, attn_kernel=kernel, kv_chunk=1024)
        step.attn(ww)
        torch.cuda.synchronize()
        assert int(step.dev_status.item()) == 0
        err = float(np.abs(step.attn_out_f32.cpu().double().numpy() - ref["attn_out"]).max())
        lse_err = float(np.abs(step.lse.cpu().double().numpy() - ref["lse"]).max())
        assert err < TOL_ATTN_F32 and lse_err < TOL_LSE, (kernel, err, lse_err)


@pytest.mark.parametrize("name,window,kv_chunk,subset", [
    ("tiny_ragged_t1", 1, 0, None), ("tiny_ragged_t1", 5, 64, None), ("tiny_ragged_t0", 40, 64, None),
    ("tiny_t1", 100, 64, None), ("tiny_t1", 1000, 0, None),
    ("qwen7b_b16_t1", 512, 0, None), ("qwen7b_b16_t1", 1500, 256, None),
    ("gemma12b_b32_t1", 1024, 0, [0, 7, 19, 31]),
])
def test_sliding_window_attention(name, window, kv_chunk, subset):
    """Local-attention variant: each block row sees only its last `window` positions.  Windows
    shorter than, comparable to and longer than the context, with automatic and forced chunking
    (whole chunks before the window are skipped; the first needed chunk starts mid-way)."""
    run_case(name, subset=subset, check_determinism=False, window=window, kv_chunk=kv_chunk)


@pytest.mark.parametrize("fused", [False, True], ids=["own_statistics", "after_accept"])
@pytest.mark.parametrize("name,subset", [("tiny_ragged_t1", None), ("tiny_peaked_t1", None), ("qwen7b_b16_t1", [0, 5, 15])])
def test_tvd_diagnostic_matches_oracle(name, subset, fused):
    """massv_tvd (Eq. 6) against the oracle's TVD of (softmax of oracle logits, q), row by row;
    1 - TVD must equal the acceptance probability output.  Tolerance 1e-4 absolute, the
    tolerance of the probabilities it is a sum of differences of.  Both forms: the stand-alone call
    that computes the rows' softmax statistics itself, and massv_tvd_after_accept, which takes them
    from the acceptance call's workspace and reads the logits once."""
    import paper_2505_10526_b200 as mv
    cfg = get_config(name)
    w = generate(cfg, device="cuda", with_attention=False)
    B, R, g, V = cfg.batch, cfg.rows, cfg.gamma, cfg.vocab
    desc = mv.accept_desc(B, g, cfg.hidden, V, cfg.temperature)
    ws = mv.alloc_workspace(mv.massv_accept_workspace_size(desc), "cuda")
    toks = torch.zeros((B, R), dtype=torch.int32, device="cuda"); lens = torch.zeros((B,), dtype=torch.int32, device="cuda")
    logits = torch.zeros((B, R, V), dtype=torch.float32, device="cuda")
    mv.massv_accept(desc, w["hidden"], w["lm_head"], w["draft_tokens"], w["draft_probs"], w["u_accept"], w["u_sample"],
                    toks, lens, logits, None, ws, None)
    tvd = torch.zeros((B, g), dtype=torch.float32, device="cuda"); acc = torch.zeros_like(tvd)
    ws2 = mv.alloc_workspace(mv.massv_tvd_workspace_size(desc), "cuda")
    if fused:
        mv.massv_tvd_after_accept(desc, logits, w["draft_probs"], ws, tvd, acc, ws2, None)
    else:
        mv.massv_tvd(desc, logits, w["draft_probs"], tvd, acc, ws2, None)
    torch.cuda.synchronize()
    idx = list(range(B)) if subset is None else subset
    hid = oracle.bf16_bits(w["hidden"])[idx].reshape(len(idx) * R, cfg.hidden)
    p = oracle.softmax(oracle.logits(hid, oracle.bf16_bits(w["lm_head"])), cfg.temperature).reshape(len(idx), R, V)
    q = w["draft_probs"].double().cpu().numpy()[idx]
    for i, b in enumerate(idx):
        for j in range(g):
            ref = oracle.tvd(np.ascontiguousarray(p[i, j]), np.ascontiguousarray(q[i, j]))
            assert abs(float(tvd[b, j]) - ref) < 1e-4, (b, j, float(tvd[b, j]), ref)
            assert abs(float(acc[b, j]) - (1.0 - ref)) < 1e-4
            assert 0.0 <= float(tvd[b, j]) <= 1.0 + 1e-6


@pytest.mark.parametrize("n,bins", [(0, 8), (1, 1), (1000, 10), (100003, 50), (3_000_000, 4096), (70001, 37)])
def test_tvd_histogram_matches_oracle(n, bins):
    """Bit-exact counts: both sides take the bin from one fp32 product.  Values are a skewed mix on [0, 1]
    with exact edges (0, 1, k / bins), strays just outside, and NaN; a second call accumulates."""
    import paper_2505_10526_b200 as mv
    gen = torch.Generator(device="cpu"); gen.manual_seed(1000 + n + bins)
    v = torch.rand((n,), generator=gen, dtype=torch.float32) ** 3            # concentrated at low values, as in Fig. 4
    if n >= 1000:
        v[:bins] = torch.arange(bins, dtype=torch.float32) / bins             # exact edges
        v[bins] = 1.0; v[bins + 1] = 0.0; v[bins + 2] = float("nan"); v[bins + 3] = 1.0000001; v[bins + 4] = -1e-8
    dv = v.cuda()
    counts = torch.zeros((bins,), dtype=torch.int64, device="cuda")
    mv.massv_tvd_histogram(dv, counts)
    torch.cuda.synchronize()
    want = oracle.tvd_histogram(v.numpy(), bins)
    assert np.array_equal(counts.cpu().numpy(), want)
    assert int(counts.sum()) == n - (1 if n >= 1000 else 0)
    mv.massv_tvd_histogram(dv, counts)
    torch.cuda.synchronize()
    assert np.array_equal(counts.cpu().numpy(), 2 * want)


def test_tvd_histogram_of_a_verify_steps_distances():
    """massv_tvd's output through massv_tvd_histogram equals the oracle's histogram of the same fp32 values,
    and of the oracle's own distances wherever those are not within 1e-4 of a bin edge."""
    import paper_2505_10526_b200 as mv
    cfg = get_config("tiny_ragged_t1")
    w = generate(cfg, device="cuda", with_attention=False)
    B, R, g, V = cfg.batch, cfg.rows, cfg.gamma, cfg.vocab
    desc = mv.accept_desc(B, g, cfg.hidden, V, cfg.temperature)
    ws = mv.alloc_workspace(mv.massv_accept_workspace_size(desc), "cuda")
    toks = torch.zeros((B, R), dtype=torch.int32, device="cuda"); lens = torch.zeros((B,), dtype=torch.int32, device="cuda")
    logits = torch.zeros((B, R, V), dtype=torch.float32, device="cuda")
    mv.massv_accept(desc, w["hidden"], w["lm_head"], w["draft_tokens"], w["draft_probs"], w["u_accept"], w["u_sample"],
                    toks, lens, logits, None, ws, None)
    tvd = torch.zeros((B, g), dtype=torch.float32, device="cuda")
    mv.massv_tvd(desc, logits, w["draft_probs"], tvd, None, mv.alloc_workspace(mv.massv_tvd_workspace_size(desc), "cuda"), None)
    bins = 8
    counts = torch.zeros((bins,), dtype=torch.int64, device="cuda")
    mv.massv_tvd_histogram(tvd, counts)
    torch.cuda.synchronize()
    assert np.array_equal(counts.cpu().numpy(), oracle.tvd_histogram(tvd.cpu().numpy(), bins))
    p = oracle.softmax(oracle.logits(oracle.bf16_bits(w["hidden"]).reshape(B * R, cfg.hidden), oracle.bf16_bits(w["lm_head"])),
                       cfg.temperature).reshape(B, R, V)
    q = w["draft_probs"].double().cpu().numpy()
    ref = np.array([[oracle.tvd(np.ascontiguousarray(p[b, j]), np.ascontiguousarray(q[b, j])) for j in range(g)] for b in range(B)])
    clear = np.abs(ref * bins - np.round(ref * bins)) > 1e-4 * bins
    got_bins = np.minimum((tvd.cpu().numpy() * np.float32(bins)).astype(np.int64), bins - 1)
    assert np.array_equal(got_bins[clear], np.minimum((ref * bins).astype(np.int64), bins - 1)[clear])
    assert int(counts.sum()) == B * g


def test_gamma_zero_sampling_is_the_draft_side_step():
    """With no drafts and T > 0 the call is one ordinary sampling step: the token is the
    inverse-CDF draw from softmax(z / T) with the caller's uniform, and probs_out is that
    distribution - which is exactly what a drafter must hand to the next verify step."""
    from dataclasses import replace
    from paper_2505_10526_b200 import VerifyStep
    cfg = replace(get_config("tiny_peaked_t1"), gamma=0, name="draft_step", batch=9, temperature=0.8)
    w = generate(cfg, device="cuda")
    step = VerifyStep.for_workload(cfg, w, want_logits=True, want_probs=True)
    ref = oracle.verify_step({k: v.clone() for k, v in w.items()}, cfg.temperature)
    step.run(w)
    torch.cuda.synchronize()
    st = compare_accept(ref, step.out_tokens.cpu().numpy(), step.accept_len.cpu().numpy(), 0)
    assert st["hard"] == 0 and np.all(step.accept_len.cpu().numpy() == 1)
    p = step.probs.cpu().double().numpy().reshape(cfg.batch, cfg.vocab)
    assert np.abs(p - ref["probs"]).max() < TOL_PROB
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-4)
    # every drawn token has positive probability and lies where the uniform points in the CDF
    toks = step.out_tokens.cpu().numpy()[:, 0]
    u = w["u_sample"].cpu().numpy()[:, 0]
    cdf = np.cumsum(ref["probs"], axis=-1)
    for b in range(cfg.batch):
        if ref["margin_sample"][b] >= 1e-3:
            assert toks[b] == int(np.searchsorted(cdf[b], u[b] * cdf[b, -1], side="right"))


def test_timing_hook_brackets_the_dominant_kernels():
    """Events handed to massv_set_timing_events are recorded around the LM-head kernel and the attention
    split kernel: both intervals are positive and lie inside the interval of the whole step; with the hook
    switched off again the events are not touched."""
    import paper_2505_10526_b200 as mv
    from paper_2505_10526_b200 import VerifyStep
    cfg = get_config("qwen7b_b1_t0")
    w = generate(cfg, device="cuda")
    step = VerifyStep.for_workload(cfg, w)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)]
    step.run(w, commit=False)                       # warm-up
    try:
        ev[0].record()
        mv.massv_set_timing_events(lm_head=(ev[1], ev[2]), attn=(ev[3], ev[4]))
        step.run(w, commit=False)
    finally:
        mv.massv_set_timing_events(None, None)
    ev[5].record()
    torch.cuda.synchronize()
    whole, lm, attn = ev[0].elapsed_time(ev[5]), ev[1].elapsed_time(ev[2]), ev[3].elapsed_time(ev[4])
    assert 0.0 < attn < whole and 0.0 < lm < whole
    assert ev[0].elapsed_time(ev[3]) >= 0.0 and ev[4].elapsed_time(ev[1]) >= 0.0 and ev[2].elapsed_time(ev[5]) >= 0.0
    assert lm > 0.1          # 1.09 GB of weights cannot be read in less than 0.1 ms
    step.run(w, commit=False)
    torch.cuda.synchronize()
    assert ev[1].elapsed_time(ev[2]) == lm          # not re-recorded once the hook is off


def _attention_only_case(cfg, kernel, kv_chunk=0, window=0):
    """massv_verify_attn alone (no LM head) against the oracle's attention, for shapes whose
    acceptance part would be out of range or beside the point."""
    from paper_2505_10526_b200 import VerifyStep
    w = generate(cfg, device="cuda")
    before = {k: w[k].clone() for k in ("k_pages", "v_pages", "seq_lens")}
    step = VerifyStep.for_workload(cfg, w, want_attn_f32=True, attn_kernel=kernel, kv_chunk=kv_chunk, window=window)
    step.attn(w)
    torch.cuda.synchronize()
    assert int(step.dev_status.item()) == 0
    # the oracle appends the block to copies of the pools as they were before the call, then attends
    kp, vp = oracle.bf16_bits(before["k_pages"]).copy(), oracle.bf16_bits(before["v_pages"]).copy()
    pt = w["page_table"].cpu().numpy().astype(np.int32)
    seq = before["seq_lens"].cpu().numpy().astype(np.int32)
    oracle.kv_append(oracle.bf16_bits(w["k_new"]), oracle.bf16_bits(w["v_new"]), kp, vp, pt, seq)
    out, lse = oracle.verify_attn(oracle.bf16_bits(w["q"]), kp, vp, pt, seq, window=window)
    ref = dict(attn_out=out, lse=lse, k_pages=kp, v_pages=vp)
    err = float(np.abs(step.attn_out_f32.cpu().double().numpy() - ref["attn_out"]).max())
    err16 = float(np.abs(step.attn_out.cpu().double().numpy() - ref["attn_out"]).max())
    lse_err = float(np.abs(step.lse.cpu().double().numpy() - ref["lse"]).max())
    _report(dict(config=cfg.name, kernel=kernel, attn_err_f32=err, attn_err_bf16=err16, lse_err=lse_err))
    assert err < TOL_ATTN_F32 and err16 < TOL_ATTN_BF16 and lse_err < TOL_LSE
    assert np.array_equal(oracle.bf16_bits(w["k_pages"]), ref["k_pages"]) and np.array_equal(oracle.bf16_bits(w["v_pages"]), ref["v_pages"])


@pytest.mark.parametrize("kernel", KERNELS)
def test_one_long_sequence_is_cut_across_many_ctas(kernel):
    """A single 20,000-token context: with the balanced schedule each (sequence, head) pair is cut
    into about sixty pieces held by consecutive CTAs, all merged by the second kernel."""
    from dataclasses import replace
    cfg = replace(get_config("qwen7b_b1_t0"), name="one_long_sequence", ctx_lo=20000, ctx_hi=20000, hidden=256, vocab=1024, seed=31)
    _attention_only_case(cfg, kernel)


@pytest.mark.parametrize("kernel", KERNELS)
def test_batch_beyond_the_balanced_schedule_limit(kernel):
    """1,100 short sequences: more than the balanced schedule indexes in shared memory, so the
    tcgen05 kernel runs on the (chunk, head, sequence) grid; lengths start at zero."""
    from workloads import VerifyConfig
    cfg = VerifyConfig(name="big_batch", batch=1100, gamma=1, n_q_heads=4, n_kv_heads=2, head_dim=64, hidden=64, vocab=64,
                       temperature=0.0, ctx_lo=0, ctx_hi=90, image_tokens=0.25, draft_noise_std=0.5, seed=77)
    _attention_only_case(cfg, kernel)


TOP_P_CASES = [
    # rows, vocab, logit scale, temperature, top_p, quantise logits (forces many exactly equal probabilities)
    (16, 1024, 2.0, 1.0, 0.9, False), (16, 1024, 2.0, 0.7, 0.5, False), (8, 1000, 4.0, 1.3, 0.25, False),
    (8, 257, 1.0, 1.0, 1.0, False), (8, 4096, 3.0, 1.0, 1e-6, False), (12, 2048, 2.0, 1.0, 0.8, True),
    (64, 152064, 1.5, 1.0, 0.95, False), (4, 152064, 6.0, 0.8, 0.5, False),
]


@pytest.mark.parametrize("rows,vocab,scale,T,top_p,quant", TOP_P_CASES)
def test_top_p_sampling_matches_oracle(rows, vocab, scale, T, top_p, quant):
    """massv_sample_top_p against the oracle's sort-based definition.  Nucleus membership (which entries
    of probs_out are non-zero) and the drawn token are exact, except where the oracle's margins say the
    decision is within rounding: the prefix mass that stops the nucleus within 1e-5 of top_p (fp32 weights
    against fp64 ones), the uniform within 1e-3 of a CDF edge; q within 1e-4 absolute."""
    import paper_2505_10526_b200 as mv
    g = torch.Generator(device="cuda"); g.manual_seed(1000 + rows + vocab)
    z = torch.randn((rows, vocab), generator=g, device="cuda", dtype=torch.float32) * scale
    if quant:
        z = torch.round(z * 2.0) / 2.0
    u = torch.rand((rows,), generator=g, device="cuda", dtype=torch.float32)
    tok = torch.full((rows,), -5, dtype=torch.int32, device="cuda")
    q = torch.full((rows, vocab), -1.0, dtype=torch.float32, device="cuda")
    status = torch.zeros((1,), dtype=torch.int32, device="cuda")
    mv.massv_sample_top_p(z, u, tok, T, top_p, q, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref = oracle.sample_top_p(z.cpu().numpy(), u.cpu().numpy(), T, top_p)
    qg, tg = q.cpu().double().numpy(), tok.cpu().numpy()
    exempt_set = exempt_draw = 0
    for r in range(rows):
        assert abs(qg[r].sum() - 1.0) < 1e-4 and qg[r].min() >= 0.0
        if ref["margin_set"][r] < 1e-5 and not np.array_equal(qg[r] > 0, ref["q"][r] > 0):
            exempt_set += 1
            continue
        # zero-probability members of the oracle's nucleus (top_p = 1 keeps everything) are not members here
        assert np.array_equal(qg[r] > 0, ref["q"][r] > 0), (r, int((qg[r] > 0).sum()), int(ref["nucleus_size"][r]))
        assert np.abs(qg[r] - ref["q"][r]).max() < TOL_PROB
        if tg[r] != ref["token"][r]:
            assert ref["margin_sample"][r] < 1e-3, (r, int(tg[r]), int(ref["token"][r]), float(ref["margin_sample"][r]))
            exempt_draw += 1
        assert qg[r][tg[r]] > 0
    _report(dict(config=f"top_p rows={rows} V={vocab} T={T} p={top_p} quant={quant}", exempt_set=exempt_set, exempt_draw=exempt_draw))
    assert exempt_set <= max(1, rows // 8)
    # a second run is bit-identical
    tok2 = torch.empty_like(tok); q2 = torch.empty_like(q)
    mv.massv_sample_top_p(z, u, tok2, T, top_p, q2, status)
    torch.cuda.synchronize()
    assert torch.equal(tok, tok2) and torch.equal(q, q2)


def test_top_p_output_feeds_the_acceptance_call():
    """Drafter-side chain: logits from massv_accept (gamma = 0 rows), massv_sample_top_p for the drafts and
    their distribution q, and q accepted as draft_probs by massv_accept: a drafter identical to the target
    (same logits, T = 1, top_p = 1) has every draft accepted, since min(1, p/q) = 1."""
    import paper_2505_10526_b200 as mv
    cfg = get_config("tiny_peaked_t1")
    w = generate(cfg, device="cuda", with_attention=False)
    B, R, g, V = cfg.batch, cfg.rows, cfg.gamma, cfg.vocab
    desc = mv.accept_desc(B, g, cfg.hidden, V, 1.0)
    ws = mv.alloc_workspace(mv.massv_accept_workspace_size(desc), "cuda")
    toks = torch.zeros((B, R), dtype=torch.int32, device="cuda"); lens = torch.zeros((B,), dtype=torch.int32, device="cuda")
    logits = torch.zeros((B, R, V), dtype=torch.float32, device="cuda")
    mv.massv_accept(desc, w["hidden"], w["lm_head"], w["draft_tokens"], w["draft_probs"], w["u_accept"], w["u_sample"],
                    toks, lens, logits, None, ws, None)
    z_draft = logits[:, :g].contiguous().view(B * g, V)
    u = torch.rand((B * g,), device="cuda", dtype=torch.float32)
    d_tok = torch.zeros((B * g,), dtype=torch.int32, device="cuda")
    d_q = torch.zeros((B * g, V), dtype=torch.float32, device="cuda")
    mv.massv_sample_top_p(z_draft, u, d_tok, 1.0, 1.0, d_q, None)
    mv.massv_accept(desc, w["hidden"], w["lm_head"], d_tok.view(B, g).contiguous(), d_q.view(B, g, V), w["u_accept"], w["u_sample"],
                    toks, lens, None, None, ws, None)
    torch.cuda.synchronize()
    # u * q < p fails only if rounding puts q above p by more than a factor 1/u: u is below 0.999 here
    assert float(w["u_accept"].max()) < 0.9999
    assert torch.all(lens == R) and torch.equal(toks[:, :g], d_tok.view(B, g))


@pytest.mark.parametrize("name", ["tiny_ragged_t1", "tiny_ragged_t0"])
def test_host_staged_step_equals_the_device_resident_step(name):
    """VerifyStep.run_host (inputs from pinned host memory, results to pinned host memory) returns what
    the device-resident step returns, with the single staging buffer and with separate host tensors."""
    from paper_2505_10526_b200 import VerifyStep
    from paper_2505_10526_b200.step import STEP_INPUTS
    cfg = get_config(name)
    w = generate(cfg, device="cuda")
    seq0 = w["seq_lens"].clone()
    ref = VerifyStep.for_workload(cfg, w)
    ref.run(w, commit=False)
    torch.cuda.synchronize()
    keys = [k for k in STEP_INPUTS if k in w and (cfg.temperature > 0 or k not in ("draft_probs", "u_accept", "u_sample"))]
    resident = {k: w[k] for k in ("k_pages", "v_pages", "page_table", "seq_lens", "lm_head")}
    one = VerifyStep.for_workload(cfg, w)
    views = one.host_inputs_like({k: w[k].cpu() for k in keys})
    toks, lens = one.run_host(views, resident, commit=False)
    assert torch.equal(toks, ref.out_tokens.cpu()) and torch.equal(lens, ref.accept_len.cpu())
    assert one.host_bytes_per_step(views)[0] >= sum(w[k].numel() * w[k].element_size() for k in keys)
    many = VerifyStep.for_workload(cfg, w)
    toks2, lens2 = many.run_host({k: w[k].cpu().pin_memory() for k in keys}, resident, commit=False)
    assert torch.equal(toks2, ref.out_tokens.cpu()) and torch.equal(lens2, ref.accept_len.cpu())
    assert torch.equal(w["seq_lens"], seq0)


@pytest.mark.parametrize("seed", range(24))
def test_attention_on_random_small_shapes(seed):
    """Seeded random geometry: heads, group size, head_dim, gamma, context ranges that start at zero,
    sliding windows and forced chunk sizes, each through both split kernels."""
    import random
    from workloads import VerifyConfig
    rnd = random.Random(9000 + seed)
    d = rnd.choice([64, 128, 128, 256])
    gamma = rnd.randint(0, 7)
    n_kv = rnd.choice([1, 2, 4])
    group = rnd.randint(1, max(1, min(8, 64 // (gamma + 1))))
    ctx_hi = rnd.choice([40, 150, 333, 700])
    cfg = VerifyConfig(name=f"fuzz{seed}", batch=rnd.randint(1, 6), gamma=gamma, n_q_heads=n_kv * group, n_kv_heads=n_kv,
                       head_dim=d, hidden=64, vocab=64, temperature=0.0, ctx_lo=rnd.choice([0, 0, ctx_hi // 2]), ctx_hi=ctx_hi,
                       image_tokens=0.25, draft_noise_std=0.5, seed=9000 + seed)
    window = rnd.choice([0, 0, 1, 17, 64, 200])
    kv_chunk = rnd.choice([0, 0, 64, 128])
    for kernel in (1, 2):
        _attention_only_case(cfg, kernel, kv_chunk=kv_chunk, window=window)


@pytest.mark.parametrize("seed", range(16))
def test_whole_step_on_random_small_shapes(seed):
    """Seeded random geometry for the whole step: vocabulary sizes off the 128-row tile, hidden sizes of
    one to nine K blocks, row counts from 1 to a few hundred (single CTAs and CTA pairs in the LM head),
    greedy and sampled verification."""
    import random
    from workloads import VerifyConfig
    rnd = random.Random(7000 + seed)
    gamma = rnd.randint(0, 7)
    batch = rnd.choice([1, 2, 3, 5, 9, 17, 40])
    while batch * (gamma + 1) > 320:
        batch //= 2
    n_kv = rnd.choice([1, 2])
    group = rnd.randint(1, max(1, min(4, 64 // (gamma + 1))))
    cfg = VerifyConfig(name=f"stepfuzz{seed}", batch=batch, gamma=gamma, n_q_heads=n_kv * group, n_kv_heads=n_kv,
                       head_dim=rnd.choice([64, 128]), hidden=64 * rnd.randint(1, 9), vocab=8 * rnd.randint(40, 1500),
                       temperature=rnd.choice([0.0, 0.0, 0.6, 1.0, 1.4]), ctx_lo=0, ctx_hi=rnd.choice([30, 120, 300]),
                       image_tokens=0.25, draft_noise_std=rnd.choice([0.3, 1.0]), seed=7000 + seed,
                       hidden_std=rnd.choice([1.0, 6.0]))
    run_case(None, cfg=cfg, check_determinism=(seed % 4 == 0))

"""The synthetic workload generator: shapes, determinism, page-table validity."""
import numpy as np
import torch

from workloads import CONFIGS, PAGE_SIZE, generate, get_config, kv_bytes


def test_tiny_workload_shapes_and_determinism():
    cfg = get_config("tiny_t1")
    a, b = generate(cfg), generate(cfg)
    for k in a:
        assert torch.equal(a[k], b[k]), k
    B, R, g = cfg.batch, cfg.rows, cfg.gamma
    assert a["q"].shape == (B, R, cfg.n_q_heads, cfg.head_dim) and a["q"].dtype == torch.bfloat16
    assert a["k_new"].shape == (B, R, cfg.n_kv_heads, cfg.head_dim)
    assert a["k_pages"].shape[1:] == (cfg.n_kv_heads, PAGE_SIZE, cfg.head_dim)
    assert a["hidden"].shape == (B, R, cfg.hidden) and a["lm_head"].shape == (cfg.vocab, cfg.hidden)
    assert a["draft_tokens"].shape == (B, g) and a["draft_probs"].shape == (B, g, cfg.vocab)
    assert int(a["seq_lens"][0]) == 256 and int(a["n_image"][0]) == 64
    np.testing.assert_allclose(a["draft_probs"].sum(-1).numpy(), 1.0, atol=1e-5)
    assert float(a["u_accept"].min()) >= 0 and float(a["u_accept"].max()) < 1
    assert kv_bytes(cfg, a["seq_lens"]) == (256 + 6) * 64 * 2 * 2


def test_page_tables_map_distinct_pages_and_cover_the_block():
    for name in ("tiny_ragged_t1", "tiny_ragged_t0", "tiny_peaked_t1"):
        cfg = get_config(name)
        w = generate(cfg)
        used = []
        for b in range(cfg.batch):
            need = (int(w["seq_lens"][b]) + cfg.rows + PAGE_SIZE - 1) // PAGE_SIZE
            row = w["page_table"][b]
            assert torch.all(row[:need] >= 0) and torch.all(row[need:] == -1)
            used += row[:need].tolist()
        assert len(used) == len(set(used)) and max(used) < w["k_pages"].shape[0]


def test_greedy_workload_has_no_draft_distribution():
    w = generate(get_config("tiny_t0"))
    assert "draft_probs" not in w and w["draft_tokens"].dtype == torch.int32


def test_config_table_covers_the_five_benchmark_shapes():
    for n in ("tiny_t0", "tiny_t1", "qwen7b_b1_t0", "qwen7b_b16_t1", "gemma12b_b32_t1",
              "qwen7b_long_g3_t0", "qwen7b_long_g5_t1", "qwen7b_long_g7_t1"):
        assert n in CONFIGS
    c = get_config("gemma12b_b32_t1")
    assert (c.n_q_heads, c.n_kv_heads, c.head_dim, c.hidden, c.vocab) == (16, 8, 256, 3840, 262144)


def test_philox_matches_the_published_known_answers():
    """Philox4x32-10 known-answer vectors (Salmon et al., SC 2011, the reference test vectors of the algorithm):
    counter and key all zero, all ones, and the digits of pi."""
    from workloads.philox import philox4x32_10, uniforms
    cases = [([0, 0, 0, 0], (0, 0), [0x6627e8d5, 0xe169c58d, 0xbc57ac4c, 0x9b00dbd8]),
             ([0xffffffff] * 4, (0xffffffff, 0xffffffff), [0x408f276d, 0x41c83b0e, 0xa20bc7c6, 0x6d5451fd]),
             ([0x243f6a88, 0x85a308d3, 0x13198a2e, 0x03707344], (0xa4093822, 0x299f31d0),
              [0xd16cfe09, 0x94fdcceb, 0x5001e420, 0x24126ea1])]
    for counter, key, want in cases:
        got = philox4x32_10(np.array([counter], dtype=np.uint32), key)[0]
        assert got.tolist() == want
    u = uniforms(100003, 7, 1)
    assert u.dtype == np.float32 and u.min() >= 0.0 and u.max() < 1.0 and abs(float(u.mean()) - 0.5) < 5e-3
    assert np.array_equal(u[:10], uniforms(10, 7, 1)) and not np.array_equal(u[:10], uniforms(10, 7, 0)[:10])


def test_uniforms_do_not_depend_on_the_device_the_workload_is_built_on():
    from workloads.philox import uniforms
    cfg = get_config("tiny_t1")
    w = generate(cfg)
    assert np.array_equal(w["u_accept"].numpy().ravel(), uniforms(cfg.batch * cfg.gamma, cfg.seed, 0))
    assert np.array_equal(w["u_sample"].numpy().ravel(), uniforms(cfg.batch * cfg.rows, cfg.seed, 1))

"""Vocabulary-sharded acceptance vs the CPU oracle of the unsharded step.

All ranks of a world run on ONE device, phase by phase (``run_lockstep``): every rank's kernels finish
before the exchange that follows them, so no kernel waits on another.  The oracle never sees a shard: it
computes the whole-vocabulary step, and the sharded result must agree with it exactly as the unsharded
kernel path does (bit-exact tokens and lengths, except at decisions whose oracle margin is below 1e-3).
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from parity_util import compare_accept, sub_workload
from workloads import generate, get_config

pytestmark = pytest.mark.gpu


def _run_sharded(cfg, w, world, transport="concat"):
    from paper_2505_10526_b200.sharded import ShardedAccept, run_lockstep
    assert cfg.vocab % world == 0
    Vs = cfg.vocab // world
    ranks = [ShardedAccept(cfg.batch, cfg.gamma, cfg.hidden, Vs, cfg.temperature, world, r) for r in range(world)]
    inputs = []
    for r in range(world):
        kw = dict(hidden=w["hidden"], lm_head_shard=w["lm_head"][r * Vs:(r + 1) * Vs].contiguous(),
                  draft_tokens=w["draft_tokens"])
        if cfg.temperature > 0:
            kw.update(draft_probs_shard=w["draft_probs"][:, :, r * Vs:(r + 1) * Vs].contiguous(),
                      u_accept=w["u_accept"], u_sample=w["u_sample"])
        inputs.append(kw)
    res = run_lockstep(ranks, inputs, transport=transport)
    torch.cuda.synchronize()
    for rk in ranks:
        assert int(rk.dev_status.item()) == 0
    toks, lens = res[0]
    for t, l in res[1:]:                       # every rank ends with the same answer
        assert torch.equal(t, toks) and torch.equal(l, lens)
    return toks, lens, ranks


def _check(cfg, world, subset=None, w=None, transport="concat"):
    w = w or generate(cfg, device="cuda", with_attention=False)
    toks, lens, ranks = _run_sharded(cfg, w, world, transport)
    idx = list(range(cfg.batch)) if subset is None else subset
    ref = oracle.verify_step(sub_workload(w, idx), cfg.temperature, want_attention=False)
    sel = torch.as_tensor(idx, device="cuda")
    st = compare_accept(ref, toks.index_select(0, sel).cpu().numpy(), lens.index_select(0, sel).cpu().numpy(), cfg.gamma)
    print(dict(config=cfg.name, world=world, **{k: v for k, v in st.items() if k != "details"}))
    assert st["hard"] == 0, st["details"]
    if cfg.temperature > 0:                    # the shards' logits are the oracle's columns
        R, V, Vs = cfg.rows, cfg.vocab, cfg.vocab // world
        z = torch.cat([rk.logits for rk in ranks], dim=1).view(cfg.batch, R, V).index_select(0, sel)
        assert float(np.abs(z.cpu().double().numpy().reshape(-1, V) - ref["logits"]).max()) < 2e-2
    return toks, lens


@pytest.mark.parametrize("world", [1, 2, 4])
@pytest.mark.parametrize("name", ["tiny_t0", "tiny_t1", "tiny_ragged_t0", "tiny_ragged_t1", "tiny_peaked_t1"])
def test_tiny_configs(name, world):
    _check(get_config(name), world)


@pytest.mark.parametrize("world", [2, 5])
@pytest.mark.parametrize("t", [0.0, 0.8])
def test_shards_of_several_chunks_with_a_ragged_last_chunk(world, t):
    """20480 * 5 / world entries per shard: 3 to 13 chunks of 4096, the last one partial."""
    cfg = replace(get_config("tiny_ragged_t1"), name=f"chunks_w{world}", vocab=20480 * 5, temperature=t, batch=6, seed=77)
    _check(cfg, world)


def test_sharded_result_equals_the_unsharded_call():
    """Same inputs through massv_accept and through four shards: identical tokens and lengths."""
    from paper_2505_10526_b200 import VerifyStep
    cfg = replace(get_config("tiny_peaked_t1"), vocab=32768, batch=8, seed=5)
    w = generate(cfg, device="cuda")
    toks, lens, _ = _run_sharded(cfg, w, 4)
    step = VerifyStep.for_workload(cfg, w)
    step.run(w, commit=False)
    torch.cuda.synchronize()
    assert torch.equal(step.accept_len, lens)
    assert torch.equal(step.out_tokens, toks)


def test_every_draft_accepted_draws_the_bonus_token_across_shards():
    """Uniforms of 0 accept every drafted token whose p is positive, so the extra token is the bonus draw
    from p itself (no residual): the walk over the shards' chunk masses of p picks it."""
    cfg = replace(get_config("tiny_t1"), batch=3, seed=9)
    w = generate(cfg, device="cuda", with_attention=False)
    w["u_accept"].zero_()
    toks, lens = _check(cfg, 2, w=w)
    assert bool((lens == cfg.gamma + 1).all())


@pytest.mark.parametrize("world", [1, 3, 8])
@pytest.mark.parametrize("name", ["tiny_ragged_t0", "tiny_ragged_t1"])
def test_own_all_gather_kernel_in_place_of_the_collective(name, world):
    """The three exchanges done by massv_shard_publish (stores into every rank's gathered buffer).
    tiny_ragged_t1 has batch 7: its token exchange is 28 bytes, the 4-byte store path."""
    cfg = get_config(name)
    cfg = replace(cfg, vocab=1024 * 3) if world == 3 else cfg
    _check(cfg, world, transport="publish")


def test_publish_places_every_rank_at_its_offset():
    from paper_2505_10526_b200 import binding as mv
    world, n = 4, 1000
    src = [torch.arange(n, dtype=torch.int32, device="cuda") + 10000 * r for r in range(world)]
    bufs = [torch.full((world * n,), -1, dtype=torch.int32, device="cuda") for _ in range(world)]
    for r in range(world):
        mv.massv_shard_publish(src[r], bufs, r)
    torch.cuda.synchronize()
    want = torch.cat(src)
    for b in bufs:
        assert torch.equal(b, want)
    with pytest.raises(ValueError):
        mv.massv_shard_publish(src[0], [bufs[0][:-4]] * world, 0)


@pytest.mark.parametrize("name,world,subset", [("qwen7b_b1_t0", 2, None), ("qwen7b_b16_t1", 4, [0, 7, 15]),
                                               ("qwen7b_b16_t1_peaked", 8, [3, 12])])
def test_full_size_vocabulary(name, world, subset):
    cfg = get_config(name)
    _check(cfg, world, subset=subset)


@pytest.mark.parametrize("seed", range(16))
def test_random_small_shapes(seed):
    """Seeded random geometry: 1 to 8 ranks, shard sizes off the 128-row tile and off the 4096-entry chunk,
    gamma 0 to 7, greedy and sampled, flat and peaked target distributions, either transport."""
    import random
    from workloads import VerifyConfig
    rnd = random.Random(9100 + seed)
    world = rnd.choice([1, 2, 3, 4, 6, 8])
    gamma = rnd.randint(0, 7)
    batch = rnd.choice([1, 2, 3, 5, 9, 17])
    shard = 8 * rnd.choice([16, 37, 100, 513, 1030])
    cfg = VerifyConfig(name=f"shardfuzz{seed}", batch=batch, gamma=gamma, n_q_heads=4, n_kv_heads=1, head_dim=64,
                       hidden=64 * rnd.randint(1, 6), vocab=shard * world, temperature=rnd.choice([0.0, 0.6, 1.0, 1.4]),
                       ctx_lo=8, ctx_hi=8, image_tokens=0.25, draft_noise_std=rnd.choice([0.3, 1.0]), seed=9100 + seed,
                       hidden_std=rnd.choice([1.0, 6.0]))
    _check(cfg, world, transport=rnd.choice(["concat", "publish"]))


@pytest.mark.parametrize("world", [1, 2, 4])
def test_empty_residual_falls_back_to_the_target_distribution(world):
    """p = q = one-hot on token 700 (a logit gap of 1024 underflows every other probability to zero, in
    fp32 and in fp64 alike), the drafted token is another one with p = q = 0: u * q < p fails, the draft is
    rejected, and max(p - q, 0) has no mass on any shard.  Both sides must then draw from p: token 700,
    whichever shard it lives on.  The unsharded call must agree too."""
    from paper_2505_10526_b200 import VerifyStep
    cfg = replace(get_config("tiny_t1"), batch=2, gamma=2, seed=3)
    w = generate(cfg, device="cuda", with_attention=False)
    V, K, hot = cfg.vocab, cfg.hidden, 700
    w["hidden"].fill_(2.0)
    w["lm_head"].zero_()
    w["lm_head"][hot].fill_(2.0)                               # z[hot] = 4 K = 1024, every other logit 0
    w["draft_probs"].zero_()
    w["draft_probs"][:, :, hot] = 1.0
    w["draft_tokens"].copy_(torch.tensor([[5, hot], [hot, 900]], dtype=torch.int32))
    ref = oracle.verify_step(w, cfg.temperature, want_attention=False)
    assert ref["accept_len"].tolist() == [1, 2]
    assert ref["out_tokens"][0, 0] == hot and ref["out_tokens"][1].tolist()[:2] == [hot, hot]
    toks, lens, _ = _run_sharded(cfg, w, world)
    assert lens.tolist() == [1, 2]
    assert int(toks[0, 0]) == hot and toks[1].tolist()[:2] == [hot, hot]
    wa = dict(w)
    wa.update(generate(cfg, device="cuda", with_lm_head=False))  # attention inputs for the whole-step object
    step = VerifyStep.for_workload(cfg, wa)
    step.run(wa, commit=False)
    torch.cuda.synchronize()
    assert torch.equal(step.accept_len, lens) and torch.equal(step.out_tokens, toks)

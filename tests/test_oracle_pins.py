"""Pins for the CPU oracle: closed forms, library routines, hand-worked cases,
brute-force enumeration and invariants fixed by Sec. 2.1 of the paper.  Each
test is chosen so that a plausible slip in the oracle (dropped term, wrong
sign/index, transposed operand, off-by-one in the causal extent) fails it.
"""
import json
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import scipy.special
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def to_bits(a):
    """float array -> bf16 bit patterns (values are rounded to bf16 first)."""
    return oracle.bf16_bits(torch.tensor(np.asarray(a), dtype=torch.float32).to(torch.bfloat16))


def from_bits(b):
    return torch.tensor(b.view(np.int16)).view(torch.bfloat16).double().numpy()


def make_paged(rng, seq_lens, R, Hq, Hkv, d, page=16, shuffle=True):
    B = len(seq_lens)
    npages = [(l + R + page - 1) // page for l in seq_lens]
    P = sum(npages) + 2
    ids = rng.permutation(P) if shuffle else np.arange(P)
    table = np.full((B, max(npages)), -1, dtype=np.int32)
    o = 0
    for b, n in enumerate(npages):
        table[b, :n] = ids[o:o + n]
        o += n
    kp = to_bits(rng.standard_normal((P, Hkv, page, d)))
    vp = to_bits(rng.standard_normal((P, Hkv, page, d)))
    q = to_bits(rng.standard_normal((B, R, Hq, d)))
    kn = to_bits(rng.standard_normal((B, R, Hkv, d)))
    vn = to_bits(rng.standard_normal((B, R, Hkv, d)))
    return dict(q=q, k_new=kn, v_new=vn, k_pages=kp, v_pages=vp, page_table=table,
                seq_lens=np.asarray(seq_lens, dtype=np.int32))


def logical_kv(w, b, n):
    """Gather positions 0..n-1 of sequence b from the pools as float64 [n, Hkv, d]."""
    page = w["k_pages"].shape[2]
    K = from_bits(w["k_pages"])
    V = from_bits(w["v_pages"])
    ks, vs = [], []
    for pos in range(n):
        pg = w["page_table"][b, pos // page]
        ks.append(K[pg, :, pos % page, :])
        vs.append(V[pg, :, pos % page, :])
    return np.stack(ks), np.stack(vs)


# ----------------------------------------------------------------------------- attention

def test_attention_matches_library_softmax_dense():
    rng = np.random.default_rng(1)
    seq_lens, R, Hq, Hkv, d = [0, 5, 16, 37], 4, 6, 2, 8
    w = make_paged(rng, seq_lens, R, Hq, Hkv, d)
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    out, lse = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    q = from_bits(w["q"])
    G = Hq // Hkv
    for b, L in enumerate(seq_lens):
        Kl, Vl = logical_kv(w, b, L + R)
        for h in range(Hq):
            s = q[b, :, h, :] @ Kl[:, h // G, :].T / math.sqrt(d)          # [R, L+R]
            mask = np.arange(L + R)[None, :] > (L + np.arange(R))[:, None]
            s = np.where(mask, -np.inf, s)
            pr = scipy.special.softmax(s, axis=-1)
            np.testing.assert_allclose(out[b, :, h, :], pr @ Vl[:, h // G, :], rtol=0, atol=1e-12)
            np.testing.assert_allclose(lse[b, :, h], scipy.special.logsumexp(s, axis=-1), rtol=0, atol=1e-12)


def test_attention_empty_prefix_first_row_returns_its_own_value():
    rng = np.random.default_rng(2)
    w = make_paged(rng, [0], 3, 2, 1, 4)
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    out, lse = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    vn = from_bits(w["v_new"])
    for h in range(2):
        np.testing.assert_allclose(out[0, 0, h], vn[0, 0, 0], atol=1e-15)


def test_attention_uniform_keys_give_causal_running_mean():
    """All keys zero => uniform weights => row j returns the mean of V over
    positions 0..L+j exactly; V = position index exposes the causal extent."""
    rng = np.random.default_rng(3)
    L, R, d = 21, 5, 4
    w = make_paged(rng, [L], R, 2, 2, d)
    w["k_pages"][:] = 0
    w["k_new"][:] = 0
    page = 16
    vals = np.zeros(from_bits(w["v_pages"]).shape)
    for pos in range(L):
        vals[w["page_table"][0, pos // page], :, pos % page, :] = pos
    w["v_pages"] = to_bits(vals)
    w["v_new"] = to_bits(np.broadcast_to((L + np.arange(R))[None, :, None, None], (1, R, 2, d)).copy())
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    out, lse = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    for j in range(R):
        n = L + j + 1
        np.testing.assert_allclose(out[0, j], (n - 1) / 2.0, atol=1e-12)
        np.testing.assert_allclose(lse[0, j], math.log(n), atol=1e-12)


def test_attention_two_positions_closed_form_with_scale():
    rng = np.random.default_rng(4)
    d = 8
    w = make_paged(rng, [1], 1, 1, 1, d)
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    q = from_bits(w["q"])[0, 0, 0]
    Kl, Vl = logical_kv(w, 0, 2)
    for scale in (1.0 / math.sqrt(d), 0.37):
        out, lse = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"], scale=scale)
        s0, s1 = scale * q @ Kl[0, 0], scale * q @ Kl[1, 0]
        w1 = 1.0 / (1.0 + math.exp(s0 - s1))
        np.testing.assert_allclose(out[0, 0, 0], w1 * Vl[1, 0] + (1 - w1) * Vl[0, 0], atol=1e-13)
        np.testing.assert_allclose(lse[0, 0, 0], math.log(math.exp(s0) + math.exp(s1)), atol=1e-13)


def test_attention_query_head_reads_its_kv_group():
    rng = np.random.default_rng(5)
    Hq, Hkv, d, L, R = 6, 3, 4, 9, 2
    w = make_paged(rng, [L], R, Hq, Hkv, d)
    v = np.zeros(from_bits(w["v_pages"]).shape)
    for g in range(Hkv):
        v[:, g] = g + 1
    w["v_pages"] = to_bits(v)
    w["v_new"] = to_bits(np.broadcast_to((np.arange(Hkv) + 1)[None, None, :, None], (1, R, Hkv, d)).copy())
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    out, _ = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    for h in range(Hq):
        np.testing.assert_allclose(out[0, :, h], h // (Hq // Hkv) + 1, atol=1e-12)


def test_attention_invariant_to_page_placement():
    rng = np.random.default_rng(6)
    seq_lens, R, Hq, Hkv, d = [33, 7], 3, 4, 2, 8
    w = make_paged(rng, seq_lens, R, Hq, Hkv, d, shuffle=False)
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    out0, lse0 = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    P = w["k_pages"].shape[0]
    perm = rng.permutation(P)                      # old page i moves to perm[i]
    kp2, vp2 = np.empty_like(w["k_pages"]), np.empty_like(w["v_pages"])
    kp2[perm], vp2[perm] = w["k_pages"], w["v_pages"]
    table2 = np.where(w["page_table"] >= 0, perm[np.maximum(w["page_table"], 0)], -1).astype(np.int32)
    out1, lse1 = oracle.verify_attn(w["q"], kp2, vp2, table2, w["seq_lens"])
    assert np.array_equal(out0, out1) and np.array_equal(lse0, lse1)


def test_append_writes_exactly_the_block_slots():
    rng = np.random.default_rng(7)
    seq_lens, R, Hkv, d = [14, 0, 31], 4, 2, 4
    w = make_paged(rng, seq_lens, R, 2, Hkv, d)
    k0, v0 = w["k_pages"].copy(), w["v_pages"].copy()
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    changed = np.zeros(k0.shape[:1] + k0.shape[2:3], dtype=bool)          # [page, slot]
    for b, L in enumerate(seq_lens):
        for j in range(R):
            pg, sl = w["page_table"][b, (L + j) // 16], (L + j) % 16
            assert np.array_equal(w["k_pages"][pg, :, sl], w["k_new"][b, j])
            assert np.array_equal(w["v_pages"][pg, :, sl], w["v_new"][b, j])
            changed[pg, sl] = True
    untouched = ~changed
    assert np.array_equal(w["k_pages"].transpose(0, 2, 1, 3)[untouched], k0.transpose(0, 2, 1, 3)[untouched])
    assert np.array_equal(w["v_pages"].transpose(0, 2, 1, 3)[untouched], v0.transpose(0, 2, 1, 3)[untouched])


# ----------------------------------------------------------------------------- logits / softmax

def test_logits_match_float64_matmul_and_orientation():
    rng = np.random.default_rng(8)
    M, K, V = 5, 48, 37
    h, W = to_bits(rng.standard_normal((M, K))), to_bits(0.02 * rng.standard_normal((V, K)))
    z = oracle.logits(h, W)
    np.testing.assert_allclose(z, from_bits(h) @ from_bits(W).T, rtol=0, atol=1e-13)
    onehot = np.zeros((1, K)); onehot[0, 11] = 1.0
    np.testing.assert_array_equal(oracle.logits(to_bits(onehot), W)[0], from_bits(W)[:, 11])


def test_softmax_temperature_closed_forms():
    z = np.array([[1.25, -0.5]])
    for T in (1.0, 0.5, 2.0):
        p = oracle.softmax(z, T)
        assert abs(p[0, 0] - 1.0 / (1.0 + math.exp(-(1.25 + 0.5) / T))) < 1e-15
    rng = np.random.default_rng(9)
    z = rng.standard_normal((3, 1000)) * 3
    p = oracle.softmax(z, 1.0)
    np.testing.assert_allclose(p, scipy.special.softmax(z, axis=-1), rtol=0, atol=1e-15)
    np.testing.assert_allclose(p.sum(-1), 1.0, atol=1e-12)
    np.testing.assert_allclose(oracle.softmax(z, 0.25), scipy.special.softmax(z * 4, axis=-1), rtol=0, atol=1e-14)


# ----------------------------------------------------------------------------- acceptance

def run_accept(T, p_rows=None, q_rows=None, drafts=None, u_accept=None, u_sample=None, z_rows=None):
    """Single-sequence helper around oracle.accept."""
    drafts = np.asarray(drafts, dtype=np.int32)[None, :]
    if T > 0:
        return oracle.accept(T, None, np.asarray(p_rows, dtype=np.float64),
                             drafts, np.asarray(q_rows, dtype=np.float32)[None],
                             np.asarray(u_accept, dtype=np.float32)[None], np.asarray(u_sample, dtype=np.float32)[None])
    return oracle.accept(0.0, np.asarray(z_rows, dtype=np.float64), None, drafts, None, None, None)


def test_hand_worked_examples():
    with open(os.path.join(GOLDEN, "accept_worked_examples.txt")) as f:
        cases = [json.loads(l) for l in f if l.strip() and not l.startswith("#")]
    assert len(cases) == 8
    for c in cases:
        if c["T"] > 0:
            r = run_accept(c["T"], c["p"], c["q"], c["drafts"], c["u_accept"], c["u_sample"])
        else:
            r = run_accept(0.0, z_rows=c["z"], drafts=c["drafts"])
        assert r["out_tokens"][0].tolist() == c["tokens"], c["name"]
        assert int(r["accept_len"][0]) == c["len"], c["name"]


def _dyadic_dist(rng, V, denom, positive=True):
    while True:
        cuts = np.sort(rng.integers(0, denom + 1, size=V - 1))
        parts = np.diff(np.concatenate([[0], cuts, [denom]]))
        if not positive or parts.min() > 0:
            return [Fraction(int(x), denom) for x in parts]


def _lcm(vals):
    out = 1
    for v in vals:
        out = out * v // math.gcd(out, v)
    return out


def _first_token_marginal(p0, q0, p1):
    """Exact output marginal of the first emitted token at gamma = 1 by driving
    the oracle with midpoint grids that align with every threshold."""
    V = len(p0)
    n_acc = _lcm([(p0[x] / q0[x]).denominator for x in range(V) if p0[x] < q0[x]] + [1])
    res = [max(p0[v] - q0[v], Fraction(0)) for v in range(V)]
    Rm = sum(res)
    cdf = np.cumsum(res)
    n_smp = _lcm([(c / Rm).denominator for c in cdf] + [1]) if Rm > 0 else 1
    assert n_acc <= 4096 and n_smp <= 65536
    p = np.array([[float(x) for x in p0], [float(x) for x in p1]])
    q = np.array([[float(x) for x in q0]], dtype=np.float32)
    # acceptance frequency per draft token
    ua = ((np.arange(n_acc) + 0.5) / n_acc).astype(np.float32)
    f_acc = np.zeros(V)
    for x in range(V):
        B = n_acc
        r = oracle.accept(1.0, None, np.tile(p, (B, 1)), np.full((B, 1), x, np.int32), np.tile(q[None], (B, 1, 1)),
                          ua[:, None].copy(), np.full((B, 2), 0.5, np.float32))
        f_acc[x] = np.mean(r["accept_len"] == 2)
        assert np.all(r["out_tokens"][r["accept_len"] == 2, 0] == x)
    # residual draw distribution (forced rejection: u_accept just below 1 on a token with p<q)
    res_dist = np.zeros(V)
    if Rm > 0:
        xr = next(x for x in range(V) if p0[x] < q0[x])
        us = ((np.arange(n_smp) + 0.5) / n_smp).astype(np.float32)
        B = n_smp
        u2 = np.stack([us, np.full(B, 0.5, np.float32)], axis=1)
        r = oracle.accept(1.0, None, np.tile(p, (B, 1)), np.full((B, 1), xr, np.int32), np.tile(q[None], (B, 1, 1)),
                          np.full((B, 1), 0.99999, np.float32), u2)
        assert np.all(r["accept_len"] == 1)
        res_dist = np.bincount(r["out_tokens"][:, 0], minlength=V) / B
    qf = np.array([float(x) for x in q0])
    marg = qf * f_acc
    marg += np.sum(qf * (1 - f_acc)) * res_dist
    return marg, f_acc


def test_rejection_sampling_is_lossless_on_16_token_vocab():
    """Sec. 2.1: the output distribution of speculative decoding equals the
    target's.  Enumerate every draft token with weight q(x) and integrate both
    uniforms on threshold-aligned grids: the marginal must be p exactly."""
    rng = np.random.default_rng(10)
    V = 16
    done = 0
    while done < 4:
        p0, q0, p1 = _dyadic_dist(rng, V, 64), _dyadic_dist(rng, V, 32), _dyadic_dist(rng, V, 64)
        try:
            marg, f_acc = _first_token_marginal(p0, q0, p1)
        except AssertionError:
            continue
        np.testing.assert_allclose(marg, [float(x) for x in p0], rtol=0, atol=1e-12)
        # acceptance probability per token is min(1, p/q)
        np.testing.assert_allclose(f_acc, [float(min(Fraction(1), a / b)) for a, b in zip(p0, q0)], atol=1e-12)
        done += 1


def test_acceptance_rate_equals_one_minus_tvd():
    """Summing min(1,p/q) over x ~ q gives sum_x min(p,q) = 1 - TVD(p,q) (Eq. 6)."""
    rng = np.random.default_rng(11)
    V, N = 16, 8192
    p = rng.dirichlet(np.ones(V)); q = rng.dirichlet(np.ones(V)).astype(np.float32)
    q = (q / q.sum()).astype(np.float32)
    ua = ((np.arange(N) + 0.5) / N).astype(np.float32)
    rate = 0.0
    for x in range(V):
        r = oracle.accept(1.0, None, np.tile(np.stack([p, p]), (N, 1)), np.full((N, 1), x, np.int32),
                          np.tile(q[None, None], (N, 1, 1)), ua[:, None].copy(), np.full((N, 2), 0.5, np.float32))
        rate += float(q[x]) * np.mean(r["accept_len"] == 2)
    assert abs(rate - (1.0 - oracle.tvd(p, q.astype(np.float64)))) < V / N


def test_two_draft_chain_second_token_follows_second_distribution():
    """gamma = 2 on a 4-token vocab: given that the first draft is accepted, the
    second emitted token is distributed as p_1; the first emitted token as p_0."""
    rng = np.random.default_rng(12)
    V = 4
    p0, p1, p2 = _dyadic_dist(rng, V, 16), _dyadic_dist(rng, V, 16), _dyadic_dist(rng, V, 16)
    q0 = q1 = [Fraction(1, 4)] * V
    n_acc = 4
    Ns = 48 * 16
    ua = (np.arange(n_acc) + 0.5) / n_acc
    us = (np.arange(Ns) + 0.5) / Ns
    rows = []
    for x1 in range(V):
        for x2 in range(V):
            for a1 in ua:
                for a2 in ua:
                    rows.append((x1, x2, a1, a2))
    rows = np.array(rows)
    first = np.zeros(V); second = np.zeros(V); w_second = 0.0
    p = np.array([[float(x) for x in r] for r in (p0, p1, p2)])
    q = np.full((2, V), 0.25, dtype=np.float32)
    for s in us:
        B = len(rows)
        r = oracle.accept(1.0, None, np.tile(p, (B, 1)), rows[:, :2].astype(np.int32).copy(), np.tile(q[None], (B, 1, 1)),
                          rows[:, 2:].astype(np.float32).copy(), np.full((B, 3), s, np.float32))
        wt = 1.0 / (len(rows) * len(us))          # q uniform => every row has the same weight
        np.add.at(first, r["out_tokens"][:, 0], wt)
        acc1 = r["accept_len"] >= 2
        np.add.at(second, r["out_tokens"][acc1, 1], wt)
        w_second += wt * acc1.sum()
    np.testing.assert_allclose(first, [float(x) for x in p0], atol=1e-12)
    np.testing.assert_allclose(second / w_second, [float(x) for x in p1], atol=1e-12)


def test_acceptance_invariants():
    rng = np.random.default_rng(13)
    B, gamma, V = 64, 5, 32
    p = rng.dirichlet(np.ones(V), size=B * (gamma + 1))
    q = rng.dirichlet(np.ones(V), size=B * gamma).astype(np.float32).reshape(B, gamma, V)
    drafts = rng.integers(0, V, size=(B, gamma)).astype(np.int32)
    ua = rng.random((B, gamma)).astype(np.float32); us = rng.random((B, gamma + 1)).astype(np.float32)
    r = oracle.accept(1.0, None, p, drafts, q, ua, us)
    n = r["accept_len"] - 1
    assert np.all((r["accept_len"] >= 1) & (r["accept_len"] <= gamma + 1))
    for b in range(B):
        assert r["out_tokens"][b, :n[b]].tolist() == drafts[b, :n[b]].tolist()
        assert 0 <= r["out_tokens"][b, n[b]] < V
        assert np.all(r["out_tokens"][b, n[b] + 1:] == -1)
        if n[b] < gamma:   # a residual draw has p > q at the drawn token
            t = r["out_tokens"][b, n[b]]
            assert p[b * (gamma + 1) + n[b], t] > q[b, n[b], t]
    # identical distributions: every draft is accepted (ratio 1, u < 1)
    q_same = p.reshape(B, gamma + 1, V)[:, :gamma].astype(np.float32)
    p_same = p.reshape(B, gamma + 1, V).copy(); p_same[:, :gamma] = q_same.astype(np.float64)
    r = oracle.accept(1.0, None, p_same.reshape(-1, V), drafts, q_same, ua, us)
    assert np.all(r["accept_len"] == gamma + 1)
    # disjoint supports: always rejected at once, extra token lies in supp(p)
    p_dis = np.zeros((B * (gamma + 1), V)); p_dis[:, :V // 2] = 2.0 / V
    q_dis = np.zeros((B, gamma, V), dtype=np.float32); q_dis[:, :, V // 2:] = 2.0 / V
    d_dis = rng.integers(V // 2, V, size=(B, gamma)).astype(np.int32)
    r = oracle.accept(1.0, None, p_dis, d_dis, q_dis, ua, us)
    assert np.all(r["accept_len"] == 1) and np.all(r["out_tokens"][:, 0] < V // 2)
    # zero draft probability at the drafted token: accepted iff the target gives it mass
    r = run_accept(1.0, [[0.5, 0.5, 0.0], [1.0, 0.0, 0.0]], [[0.0, 0.5, 0.5]], [0], [0.9], [0.3, 0.3])
    assert int(r["accept_len"][0]) == 2
    r = run_accept(1.0, [[0.0, 0.5, 0.5], [1.0, 0.0, 0.0]], [[0.0, 0.5, 0.5]], [0], [0.0], [0.3, 0.3])
    assert int(r["accept_len"][0]) == 1 and r["out_tokens"][0, 0] == 1     # p == q: falls back to p


def test_greedy_rule_margins_and_ties():
    z = np.array([[0.0, 3.0, 1.0], [2.0, 2.0, -1.0]])
    r = run_accept(0.0, z_rows=z, drafts=[1])
    assert r["out_tokens"][0].tolist() == [1, 0] and int(r["accept_len"][0]) == 2
    assert abs(r["margin_accept"][0, 0] - 2.0) < 1e-15 and r["margin_sample"][0] == 0.0


def test_sampling_margin_is_distance_to_cdf_edges():
    r = run_accept(1.0, [[0.1, 0.2, 0.3, 0.4], [0.25] * 4], [[0.4, 0.3, 0.2, 0.1]], [0], [0.3], [0.26, 0.5])
    # residual CDF edges 0.25 and 1.0, u = 0.26 -> token 3, only the lower edge can flip it
    assert abs(r["margin_sample"][0] - 0.01) < 1e-7
    assert abs(r["margin_accept"][0, 0] - abs(np.float32(0.3) - 0.25)) < 1e-7


def test_inverse_cdf_intervals_are_half_open():
    """A uniform exactly on a CDF edge belongs to the entry that starts there
    (first running sum strictly above u * total); zero-mass entries never win."""
    p = [[0.25, 0.25, 0.0, 0.5], [1.0, 0.0, 0.0, 0.0]]
    q = [[0.0, 0.0, 1.0, 0.0]]                        # residual of row 0 is p itself
    for u, tok in ((0.0, 0), (0.25, 1), (0.5, 3), (0.49999, 1), (0.999999, 3)):
        r = run_accept(1.0, p, q, [2], [0.5], [u, 0.5])
        assert int(r["accept_len"][0]) == 1 and int(r["out_tokens"][0, 0]) == tok, (u, tok)


# ----------------------------------------------------------------------------- closed loop: T = 0 equals greedy decoding

class ToyTarget:
    """A one-layer toy language model assembled from oracle pieces only:
    token -> embedding -> (q,k,v) projections -> block attention over a paged
    cache -> LM head.  Used to run speculative decoding end to end."""

    def __init__(self, seed, V=24, dm=16, Hq=4, Hkv=2, d=8, max_len=128):
        rng = np.random.default_rng(seed)
        self.V, self.dm, self.Hq, self.Hkv, self.d = V, dm, Hq, Hkv, d
        bf = lambda a: from_bits(to_bits(a))
        self.E = bf(rng.standard_normal((V, dm)))
        self.Wq = bf(rng.standard_normal((dm, Hq * d)) / math.sqrt(dm))
        self.Wk = bf(rng.standard_normal((dm, Hkv * d)) / math.sqrt(dm))
        self.Wv = bf(rng.standard_normal((dm, Hkv * d)) / math.sqrt(dm))
        self.Wo = bf(rng.standard_normal((Hq * d, dm)) / math.sqrt(Hq * d))
        self.lm = to_bits(rng.standard_normal((V, dm)))
        npg = max_len // 16
        self.table = rng.permutation(npg).astype(np.int32)[None, :]
        self.kp = np.zeros((npg, Hkv, 16, d), dtype=np.uint16)
        self.vp = np.zeros_like(self.kp)
        self.seq = np.zeros((1,), dtype=np.int32)

    def forward_block(self, tokens):
        """Append the block's K/V at seq.. and return fp64 logits [len(tokens), V]."""
        e = self.E[np.asarray(tokens)]
        R = len(tokens)
        q = to_bits((e @ self.Wq).reshape(1, R, self.Hq, self.d))
        k = to_bits((e @ self.Wk).reshape(1, R, self.Hkv, self.d))
        v = to_bits((e @ self.Wv).reshape(1, R, self.Hkv, self.d))
        oracle.kv_append(k, v, self.kp, self.vp, self.table, self.seq)
        out, _ = oracle.verify_attn(q, self.kp, self.vp, self.table, self.seq)
        hid = to_bits(out.reshape(R, -1) @ self.Wo + e)
        return oracle.logits(hid, self.lm)

    def live_cache(self):
        n = int(self.seq[0])
        pos = np.arange(n)
        return self.kp[self.table[0, pos // 16], :, pos % 16].copy(), self.vp[self.table[0, pos // 16], :, pos % 16].copy()


@pytest.mark.parametrize("gamma,seed", [(1, 0), (3, 1), (5, 2), (7, 3)])
def test_temperature_zero_speculative_decoding_equals_greedy(gamma, seed):
    n_new = 40
    # plain greedy decoding, one token per target pass
    tg = ToyTarget(seed)
    stream_g = [3]
    while len(stream_g) < n_new + 1:
        z = tg.forward_block([stream_g[-1]])
        r = oracle.accept(0.0, z, None, np.zeros((1, 0), np.int32), None, None, None)
        oracle.kv_commit(r["accept_len"], tg.seq)
        stream_g.append(int(r["out_tokens"][0, 0]))
    # speculative decoding with an unreliable drafter (right about 60% of the time)
    ts = ToyTarget(seed)
    rng = np.random.default_rng(100 + seed)
    stream_s = [3]
    lens = []
    while len(stream_s) < n_new + 1:
        t = len(stream_s)
        drafts = []
        for i in range(gamma):
            truth = stream_g[t + i] if t + i < len(stream_g) else 0
            drafts.append(truth if rng.random() < 0.6 else int(rng.integers(0, ts.V)))
        z = ts.forward_block([stream_s[-1]] + drafts)
        r = oracle.accept(0.0, z, None, np.asarray(drafts, np.int32)[None], None, None, None)
        n = int(r["accept_len"][0])
        assert 1 <= n <= gamma + 1
        oracle.kv_commit(r["accept_len"], ts.seq)
        stream_s.extend(int(x) for x in r["out_tokens"][0, :n])
        lens.append(n)
    m = min(len(stream_g), len(stream_s))
    assert stream_s[:m] == stream_g[:m]
    assert max(lens) > 1                              # drafts were accepted at least once
    # the committed part of the cache equals the never-drafted run's cache
    kg, vg = tg.live_cache()
    ks, vs = ts.live_cache()
    n = min(len(kg), len(ks))
    assert np.array_equal(kg[:n], ks[:n]) and np.array_equal(vg[:n], vs[:n])


def test_rollback_leaves_state_as_if_never_drafted():
    rng = np.random.default_rng(14)
    a, b = ToyTarget(7), ToyTarget(7)
    for t in (a, b):
        t.forward_block([1, 2, 3, 4]); t.seq += 4
    before = a.seq.copy()
    a.forward_block([5, 9, 9, 9, 9, 9])               # speculative block, then rolled back
    oracle.kv_commit(None, a.seq)
    assert np.array_equal(a.seq, before)
    za = a.forward_block([5, 6, 7])
    zb = b.forward_block([5, 6, 7])
    assert np.array_equal(za, zb)
    acc = np.array([2], np.int32)
    oracle.kv_commit(acc, a.seq)
    assert int(a.seq[0]) == int(before[0]) + 2


# ----------------------------------------------------------------------------- workload statistics

def test_flat_vocab_acceptance_rate_matches_gaussian_closed_form():
    """With q = softmax(z + N(0,1)) on a flat, large vocabulary the per-position
    acceptance sum_v min(p,q) tends to 2*Phi(-1/2) = 0.617.  Checks the oracle's
    measured rate on the tiny T=1 workload against sum min(p,q) per row."""
    from workloads import generate, get_config
    cfg = get_config("tiny_t1")
    w = generate(cfg)
    res = oracle.verify_step(w, cfg.temperature)
    p = res["probs"].reshape(cfg.batch, cfg.rows, -1)[:, :cfg.gamma]
    q = w["draft_probs"].double().numpy()
    exp_rate = np.minimum(p, q).sum(-1)
    assert abs(exp_rate.mean() - 2 * 0.5 * math.erfc(0.5 / math.sqrt(2))) < 0.05
    assert 1 <= int(res["accept_len"][0]) <= cfg.rows


# ----------------------------------------------------------------------------- sliding-window attention

def test_window_matches_library_softmax_with_band_mask():
    rng = np.random.default_rng(31)
    seq_lens, R, Hq, Hkv, d = [0, 5, 16, 37], 4, 4, 2, 8
    w = make_paged(rng, seq_lens, R, Hq, Hkv, d)
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    q = from_bits(w["q"])
    G = Hq // Hkv
    for window in (1, 3, 7, 100):
        out, lse = oracle.verify_attn(w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"], window=window)
        for b, L in enumerate(seq_lens):
            Kl, Vl = logical_kv(w, b, L + R)
            pos = np.arange(L + R)[None, :]
            row_pos = (L + np.arange(R))[:, None]
            hidden = (pos > row_pos) | (pos < row_pos - window + 1)
            for h in range(Hq):
                s = q[b, :, h, :] @ Kl[:, h // G, :].T / math.sqrt(d)
                s = np.where(hidden, -np.inf, s)
                pr = scipy.special.softmax(s, axis=-1)
                np.testing.assert_allclose(out[b, :, h, :], pr @ Vl[:, h // G, :], rtol=0, atol=1e-12)
                np.testing.assert_allclose(lse[b, :, h], scipy.special.logsumexp(s, axis=-1), rtol=0, atol=1e-12)


def test_window_closed_forms():
    """Window 1: every row returns its own value.  Zero keys: the mean of V over the last
    `window` positions.  A window at least as long as the context is full attention."""
    rng = np.random.default_rng(32)
    L, R, d = 21, 5, 4
    w = make_paged(rng, [L], R, 2, 2, d)
    w["k_pages"][:] = 0
    w["k_new"][:] = 0
    vals = np.zeros(from_bits(w["v_pages"]).shape)
    for pos in range(L):
        vals[w["page_table"][0, pos // 16], :, pos % 16, :] = pos
    w["v_pages"] = to_bits(vals)
    w["v_new"] = to_bits(np.broadcast_to((L + np.arange(R))[None, :, None, None], (1, R, 2, d)).copy())
    oracle.kv_append(w["k_new"], w["v_new"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    args = (w["q"], w["k_pages"], w["v_pages"], w["page_table"], w["seq_lens"])
    out1, _ = oracle.verify_attn(*args, window=1)
    out6, lse6 = oracle.verify_attn(*args, window=6)
    full, lse_full = oracle.verify_attn(*args)
    wide, lse_wide = oracle.verify_attn(*args, window=L + R)
    for j in range(R):
        np.testing.assert_allclose(out1[0, j], L + j, atol=1e-12)
        np.testing.assert_allclose(out6[0, j], L + j - 2.5, atol=1e-12)        # mean of the last six positions
        np.testing.assert_allclose(lse6[0, j], math.log(6), atol=1e-12)
    assert np.array_equal(full, wide) and np.array_equal(lse_full, lse_wide)


def test_tvd_hand_values():
    """Eq. 6 on values worked by hand: identical -> 0, disjoint -> 1, and a three-token case."""
    a = np.array([0.5, 0.3, 0.2]); b = np.array([0.2, 0.5, 0.3])
    assert abs(oracle.tvd(a, b) - 0.3) < 1e-15            # (0.3 + 0.2 + 0.1) / 2
    assert oracle.tvd(a, a.copy()) == 0.0
    assert abs(oracle.tvd(np.array([1.0, 0.0, 0.0]), np.array([0.0, 0.25, 0.75])) - 1.0) < 1e-15
    assert abs(oracle.tvd(a, b) - oracle.tvd(b, a)) < 1e-18


def test_tvd_histogram_hand_values_and_library_histogram():
    """Fig. 4's histogram of Eq. 6 values: hand-placed values, the closed right edge, accumulation over
    calls, NaN skipped, and agreement with numpy's histogram on values away from the bin edges."""
    vals = np.array([0.0, 0.049, 0.05, 0.5, 0.99, 1.0, 0.31, 0.31, np.nan], dtype=np.float32)
    c = oracle.tvd_histogram(vals, 10)
    assert c.tolist() == [3, 0, 0, 2, 0, 1, 0, 0, 0, 2]          # 0, .049, .05 | .31 x2 | .5 | .99 and 1.0
    assert c.sum() == 8                                          # the NaN is not counted
    c2 = oracle.tvd_histogram(np.array([0.05, 0.95], np.float32), 10, counts=c.copy())
    assert c2.tolist() == [4, 0, 0, 2, 0, 1, 0, 0, 0, 3]         # accumulates
    assert oracle.tvd_histogram(np.array([-1e-7, 1.0000001], np.float32), 4).tolist() == [1, 0, 0, 1]   # rounding strays
    rng = np.random.default_rng(3)
    for bins in (7, 20, 64):
        # mid-points of a fine grid: at least 1/(2*4096*bins) away from every edge, far beyond fp32 rounding
        k = rng.integers(0, 4096 * bins, size=5000)
        v = ((k + 0.5) / (4096 * bins)).astype(np.float32)
        want, _ = np.histogram(v.astype(np.float64), bins=bins, range=(0.0, 1.0))
        assert np.array_equal(oracle.tvd_histogram(v, bins), want)
    # a skewed sample keeps its shape: every TVD of identical distributions lands in bin 0
    p = rng.dirichlet(np.ones(32), size=50)
    t = np.array([oracle.tvd(p[i], p[i].copy()) for i in range(50)], np.float32)
    assert oracle.tvd_histogram(t, 16)[0] == 50


# ---------------------------------------------------------------- nucleus (top-p) sampling (Sec. 3.2)
def _softmax64(z, T):
    z = z.astype(np.float64) / T
    e = np.exp(z - z.max(-1, keepdims=True))
    return e / e.sum(-1, keepdims=True)


def test_top_p_hand_worked_example():
    """p = (0.5, 0.2, 0.2, 0.1), top_p = 0.6: the prefix (0.5, then the first of the two 0.2s) reaches 0.7,
    so the nucleus is {0, 1} (the tie goes to the lower index) and q = (5/7, 2/7, 0, 0)."""
    z = np.log(np.array([[0.5, 0.2, 0.2, 0.1]] * 3, dtype=np.float64)).astype(np.float32)
    u = np.array([0.70, 0.72, 0.0], dtype=np.float32)
    r = oracle.sample_top_p(z, u, 1.0, 0.6)
    assert r["nucleus_size"].tolist() == [2, 2, 2]
    np.testing.assert_allclose(r["q"][0], [5 / 7, 2 / 7, 0, 0], atol=1e-7)
    assert r["token"].tolist() == [0, 1, 0]          # 5/7 = 0.714: u = 0.70 falls in token 0, u = 0.72 in token 1
    np.testing.assert_allclose(r["margin_set"], 0.1, atol=1e-6)      # 0.6 is 0.1 from both 0.5 and 0.7
    # top_p = 0.7 is reached exactly by the same prefix (>=); 0.71 needs the second 0.2 as well
    assert oracle.sample_top_p(z[:1], u[:1], 1.0, 0.7 - 1e-9)["nucleus_size"][0] == 2
    assert oracle.sample_top_p(z[:1], u[:1], 1.0, 0.71)["nucleus_size"][0] == 3


def test_top_p_against_a_stable_argsort_reference():
    """Independent formulation with numpy: stable argsort of -p, cumulative sum, cut, renormalise,
    searchsorted on the vocabulary-order CDF."""
    rng = np.random.default_rng(5)
    for V, T, top_p in [(16, 1.0, 0.5), (257, 0.7, 0.9), (1000, 1.3, 0.25), (64, 1.0, 0.999)]:
        z = (rng.standard_normal((12, V)) * 2.0).astype(np.float32)
        u = rng.random(12).astype(np.float32)
        r = oracle.sample_top_p(z, u, T, top_p)
        p = _softmax64(z, T)
        for i in range(12):
            order = np.argsort(-p[i], kind="stable")
            cum = np.cumsum(p[i][order])
            k = int(np.searchsorted(cum, top_p, side="left")) + 1          # first prefix with mass >= top_p
            keep = np.zeros(V, dtype=bool); keep[order[:k]] = True
            q = np.where(keep, p[i], 0.0); q /= q.sum()
            assert r["nucleus_size"][i] == k
            np.testing.assert_allclose(r["q"][i], q, atol=1e-12)
            if r["margin_sample"][i] > 1e-9:
                assert r["token"][i] == int(np.searchsorted(np.cumsum(q), u[i] * 1.0, side="right"))
            # the nucleus is minimal: without its least likely member the mass is below top_p
            assert p[i][keep].sum() >= top_p - 1e-12 and p[i][keep].sum() - p[i][order[k - 1]] < top_p


def test_top_p_limits():
    """top_p = 1 keeps every token and is plain inverse-CDF sampling of softmax(z / T); a top_p below the
    largest probability keeps only the argmax."""
    rng = np.random.default_rng(6)
    z = (rng.standard_normal((8, 50)) * 3.0).astype(np.float32)
    u = rng.random(8).astype(np.float32)
    full = oracle.sample_top_p(z, u, 0.8, 1.0)
    p = _softmax64(z, 0.8)
    assert np.all(full["nucleus_size"] == 50)
    np.testing.assert_allclose(full["q"], p, atol=1e-12)
    for i in range(8):
        if full["margin_sample"][i] > 1e-9:
            assert full["token"][i] == int(np.searchsorted(np.cumsum(p[i]), u[i] * p[i].sum(), side="right"))
    greedy = oracle.sample_top_p(z, u, 0.8, 1e-6)
    assert np.all(greedy["nucleus_size"] == 1) and np.array_equal(greedy["token"], p.argmax(-1))


def test_top_p_marginal_is_the_renormalised_nucleus():
    """Over a fine grid of uniforms the drawn tokens follow q (grid error at most 1/N per token) and
    tokens outside the nucleus never appear."""
    rng = np.random.default_rng(7)
    z = (rng.standard_normal((1, 12)) * 1.5).astype(np.float32)
    N = 4000
    u = ((np.arange(N) + 0.5) / N).astype(np.float32)
    r = oracle.sample_top_p(np.repeat(z, N, axis=0), u, 1.0, 0.8)
    q = r["q"][0]
    freq = np.bincount(r["token"], minlength=12) / N
    assert np.all(np.abs(freq - q) <= 1.0 / N + 1e-12)
    assert np.all(freq[q == 0] == 0)

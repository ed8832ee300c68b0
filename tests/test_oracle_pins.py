"""Pins for the CPU oracle: what the paper and the mathematics fix, never the oracle's own formulas.

Hand-worked values (tests/golden), brute force over subsets, closed forms,
invariants and reductions to textbook routines (plain top-k MoE of Eq. 2, one
SwiGLU FFN, a dense softmax mixture).  No GPU needed.
"""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "handworked_routing.json")


def tiny_inputs(seed=0, M=15, cfg=None):
    cfg = cfg or synth.CONFIGS["tiny"]
    L = synth.gen_layer(cfg, seed)
    H = synth.gen_hidden(cfg, M, seed)
    f64 = lambda t: t.double().numpy()
    return cfg, f64(H), {k: f64(v) for k, v in L.items()}


def run(cfg, H, L, B, policy=orc.SUBSTITUTION, mode=orc.FROM_ALL, renorm=True, k=None, **kw):
    return orc.verify_layer(H, L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"],
                            cfg.k if k is None else k, B, policy, mode, renorm, **kw)


# ------------------------------------------------------------ hand-worked fixture
def test_handworked_routing_example():
    g = json.load(open(GOLD))
    z = np.log(np.array(g["softmax_weights"], dtype=np.float64)).astype(np.float32)
    for case in g["cases"]:
        for pol_name, pol in (("substitution", orc.SUBSTITUTION), ("truncation", orc.TRUNCATION)):
            for renorm in (True, False):
                r = orc.route(z, g["k"], case["B"], pol, orc.FROM_ALL, renorm)
                np.testing.assert_allclose(r["prob"], g["prob"], rtol=0, atol=1e-7)
                np.testing.assert_allclose(r["score"], g["score"], rtol=0, atol=1e-7)
                assert r["topk"] == g["topk"] and r["union"] == g["union"] and r["natcnt"] == g["natcnt"]
                assert r["S"] == case["S"]
                assert abs(r["coverage"] - case["coverage"]) < 1e-7
                exp = case[pol_name]
                assert r["assign"] == exp["assign"]
                np.testing.assert_allclose(r["wgt"], exp["wgt_renorm" if renorm else "wgt_raw"], rtol=0, atol=1e-7)
                assert r["count"] == exp["count"] and r["offset"] == exp["offset"]
                assert r["perm_row2tok"] == exp["perm_row2tok"]


def test_handworked_ffn_example():
    g = json.load(open(GOLD))["ffn"]
    y = orc.expert_ffn(np.array([g["x"]]), np.array(g["w_gate"]), np.array(g["w_up"]), np.array(g["w_down"]))
    np.testing.assert_allclose(y[0], g["y"], rtol=1e-15)


# ------------------------------------------------------------ O1 logits
def test_logits_against_exactly_rounded_sums():
    cfg, H, L = tiny_inputs()
    z = orc.router_logits(H, L["router_w"], L["router_bias"])
    assert z.dtype == np.float32
    for t in (0, 7, 14):
        for i in (0, 5, 15):
            exact = math.fsum([float(a) * float(b) for a, b in zip(L["router_w"][i], H[t])] + [float(L["router_bias"][i])])
            assert abs(float(z[t, i]) - exact) <= abs(exact) * 2 ** -23 + 1e-30


def test_logits_unit_vector_router_and_no_bias():
    rng = np.random.default_rng(0)
    H = rng.standard_normal((5, 8))
    Wr = np.eye(8)[[3, 0, 6]]                      # rows are unit vectors: z[t,i] = h[t, col_i]
    z = orc.router_logits(H, Wr, None)
    np.testing.assert_array_equal(z, H[:, [3, 0, 6]].astype(np.float32))
    zb = orc.router_logits(H, Wr, np.array([1.0, 0.0, -2.0]))
    np.testing.assert_allclose(zb, (H[:, [3, 0, 6]] + [1.0, 0.0, -2.0]).astype(np.float32), rtol=1e-7)


# ------------------------------------------------------------ O2 softmax
def test_softmax_invariants():
    rng = np.random.default_rng(1)
    z = (rng.standard_normal((6, 16)) * 3).astype(np.float32)
    p = orc.softmax_rows(z)
    np.testing.assert_allclose(p.sum(axis=1), 1.0, rtol=0, atol=1e-15)
    assert np.all(p > 0)
    # shift invariance with a shift that is exact in fp32
    zs = z.astype(np.float64) + 4.0
    np.testing.assert_allclose(orc.softmax_rows(zs), p, rtol=1e-15)
    np.testing.assert_array_equal(orc.softmax_rows(np.full((2, 8), 0.37, np.float32)), np.full((2, 8), 0.125))
    # ratio form of Eq. 1: p_i / p_j = exp(z_i - z_j)
    assert abs(p[2, 3] / p[2, 5] - math.exp(float(z[2, 3]) - float(z[2, 5]))) < 1e-12 * p[2, 3] / p[2, 5] + 1e-15
    # library cross-check
    ref = torch.softmax(torch.from_numpy(z).double(), dim=1).numpy()
    np.testing.assert_allclose(p, ref, rtol=1e-13)


# ------------------------------------------------------------ O3 / O6 rankings
def beats(keys, i, j):
    """i is ranked strictly before j under (key desc, index asc)."""
    return keys[i] > keys[j] or (keys[i] == keys[j] and i < j)


def test_topk_is_the_unique_dominating_set_with_ties():
    rng = np.random.default_rng(2)
    z = rng.integers(-2, 3, size=(40, 7)).astype(np.float32)      # many exact ties
    for k in (1, 3, 7, 9):
        T, union, natcnt = orc.natural_topk(z, k)
        for t in range(z.shape[0]):
            sel = T[t]
            assert len(sel) == min(k, 7) and len(set(sel)) == len(sel)
            rest = [j for j in range(7) if j not in sel]
            assert all(beats(z[t], i, j) for i in sel for j in rest)
            assert all(beats(z[t], sel[a], sel[a + 1]) for a in range(len(sel) - 1))
        assert union == sorted(set(i for s in T for i in s))
        assert natcnt == [sum(i in s for s in T) for i in range(7)]
        assert sum(natcnt) == z.shape[0] * min(k, 7)


def test_topk_matches_stable_argsort():
    rng = np.random.default_rng(3)
    z = rng.standard_normal((20, 16)).astype(np.float32)
    z[:, 4] = z[:, 9]                                              # a column-wide tie
    T, _, _ = orc.natural_topk(z, 4)
    ref = np.argsort(-z.astype(np.float64), axis=1, kind="stable")[:, :4]
    assert T == ref.tolist()


def test_substitution_and_truncation_set_relations():
    cfg, H, L = tiny_inputs()
    for B in (1, 2, 4, 8, 12, 16):
        rs = run(cfg, H, L, B, orc.SUBSTITUTION)
        rt = run(cfg, H, L, B, orc.TRUNCATION)
        S = set(rs["S"])
        assert rs["S"] == rt["S"]
        for t in range(H.shape[0]):
            Tk, As, At = set(rs["topk"][t]), rs["assign"][t], rt["assign"][t]
            assert set(At) == Tk & S                               # Eq. 7
            assert set(As) <= S and len(As) == min(cfg.k, len(S))  # Eq. 8: exactly k inside S
            assert set(As) >= Tk & S                               # surviving natural experts are kept
            rest = [j for j in S if j not in As]
            assert all(beats(rs["logits"][t], i, j) for i in As for j in rest)
            if Tk <= S:                                            # policies coincide
                assert set(As) == Tk
                np.testing.assert_array_equal(rs["wgt"][t], rt["wgt"][t])


# ------------------------------------------------------------ O4 scores
def test_scores_closed_forms():
    cfg, H, L = tiny_inputs()
    r = run(cfg, H, L, 8)
    assert abs(r["score"].sum() - H.shape[0]) < 1e-12              # each softmax row sums to 1
    Hsame = np.repeat(H[3:4], 6, axis=0)
    r2 = run(cfg, Hsame, L, 8)
    np.testing.assert_allclose(r2["score"], 6 * r2["prob"][0], rtol=1e-15)
    # column sums by an independent exactly-rounded route
    for i in (0, 7):
        assert abs(r["score"][i] - math.fsum(r["prob"][:, i])) < 1e-14


def test_coverage_monotone_in_budget():
    cfg, H, L = tiny_inputs()
    cov = [run(cfg, H, L, B)["coverage"] for B in range(1, 17)]
    assert all(0 < c <= 1 + 1e-12 for c in cov)
    assert all(b >= a for a, b in zip(cov, cov[1:]))
    assert abs(cov[-1] - 1.0) < 1e-12


# ------------------------------------------------------------ O5 shortlist
def test_shortlist_brute_force_over_subsets():
    rng = np.random.default_rng(4)
    for trial in range(30):
        N = int(rng.integers(2, 9))
        s = rng.integers(0, 4, size=N).astype(np.float64) / 4.0 if trial % 2 else rng.random(N)
        for B in range(1, N + 1):
            best = max(itertools.combinations(range(N), B),
                       key=lambda c: (sum(s[i] for i in c), tuple(-i for i in c)))
            assert sorted(orc.shortlist(s, B, range(N))) == list(best)


def test_shortlist_nesting_and_sizes_both_modes():
    cfg, H, L = tiny_inputs()
    prev = {orc.FROM_ALL: [], orc.FROM_UNION: []}
    for B in range(1, 20):
        for mode in (orc.FROM_ALL, orc.FROM_UNION):
            r = run(cfg, H, L, B, mode=mode)
            S, E = r["S"], r["union"]
            if mode == orc.FROM_ALL:
                assert len(S) == min(B, cfg.n_experts)
            else:
                assert len(S) == min(B, len(E)) and set(S) <= set(E)
            assert S[:len(prev[mode])] == prev[mode]               # S_B is a prefix of S_{B+1}
            prev[mode] = S


def test_shortlist_tie_goes_to_lower_index():
    # identical router rows give identical logits, probabilities and scores in any arithmetic
    cfg, H, L = tiny_inputs()
    L = dict(L)
    L["router_w"] = L["router_w"].copy(); L["router_bias"] = L["router_bias"].copy()
    L["router_w"][11] = L["router_w"][2]; L["router_bias"][11] = L["router_bias"][2]
    r = run(cfg, H, L, 16)
    assert r["score"][2] == r["score"][11]
    pos = r["S"].index(2)
    assert r["S"][pos + 1] == 11
    r1 = run(cfg, H, L, pos + 1)
    assert 2 in r1["S"] and 11 not in r1["S"]


# ------------------------------------------------------------ O7 weights
def test_gate_weight_sums():
    cfg, H, L = tiny_inputs()
    for B in (2, 4, 8):
        rs = run(cfg, H, L, B, orc.SUBSTITUTION, renorm=True)
        np.testing.assert_allclose(rs["wgt"].sum(axis=1), 1.0, rtol=0, atol=1e-15)
        rt = run(cfg, H, L, B, orc.TRUNCATION, renorm=True)
        p = rt["prob"]
        for t in range(H.shape[0]):
            Tk, At = rt["topk"][t], rt["assign"][t]
            want = sum(p[t, i] for i in At) / sum(p[t, i] for i in Tk)
            assert abs(rt["wgt"][t].sum() - want) < 1e-15
            assert rt["wgt"][t].sum() <= 1 + 1e-15
            assert (abs(rt["wgt"][t].sum() - 1) < 1e-15) == (set(Tk) <= set(rt["S"]))
        for pol in (orc.SUBSTITUTION, orc.TRUNCATION):
            rr = run(cfg, H, L, B, pol, renorm=False)
            mask = rr["wgt"] != 0
            np.testing.assert_array_equal(rr["wgt"][mask], rr["prob"][mask])
            assert [sorted(np.nonzero(mask[t])[0].tolist()) for t in range(H.shape[0])] == [sorted(a) for a in rr["assign"]]


# ------------------------------------------------------------ O8 layer value
def plain_topk_moe(H, L, k, renorm):
    """Eq. 2 written separately, token by token with vector operations."""
    M, d = H.shape
    out = np.zeros((M, d))
    for t in range(M):
        z = (L["router_w"] @ H[t] + L["router_bias"]).astype(np.float32).astype(np.float64)
        g = np.exp(z - z.max()); g /= g.sum()
        top = np.argsort(-z, kind="stable")[:k]
        w = g[top] / g[top].sum() if renorm else g[top]
        for wi, i in sorted(zip(w, top), key=lambda x: x[1]):
            a = L["w_gate"][i] @ H[t]; u = L["w_up"][i] @ H[t]
            silu = torch.nn.functional.silu(torch.from_numpy(a)).numpy()
            out[t] += wi * (L["w_down"][i] @ (silu * u))
    return out


@pytest.mark.parametrize("renorm", [True, False])
def test_unbudgeted_reduces_to_plain_topk_moe(renorm):
    cfg, H, L = tiny_inputs()
    ref = plain_topk_moe(H, L, cfg.k, renorm)
    scale = np.abs(ref).max()
    for pol in (orc.SUBSTITUTION, orc.TRUNCATION):
        full = run(cfg, H, L, cfg.n_experts, pol, renorm=renorm)
        np.testing.assert_allclose(full["out"], ref, rtol=0, atol=1e-12 * scale)
        over = run(cfg, H, L, cfg.n_experts + 5, pol, renorm=renorm)
        np.testing.assert_array_equal(over["out"], full["out"])
        # union reading: any B >= |E| reproduces the unbudgeted layer exactly
        nE = len(full["union"])
        ru = run(cfg, H, L, nE, pol, mode=orc.FROM_UNION, renorm=renorm)
        assert sorted(ru["S"]) == full["union"]
        np.testing.assert_array_equal(ru["out"], full["out"])


def test_shortlist_containing_union_is_unbudgeted():
    cfg, H, L = tiny_inputs(M=3)
    full = run(cfg, H, L, cfg.n_experts)
    for B in range(1, cfg.n_experts + 1):
        r = run(cfg, H, L, B)
        if set(r["S"]) >= set(r["union"]):
            np.testing.assert_array_equal(r["out"], full["out"])
            break
    else:
        pytest.fail("no budget contained the union")


def test_single_token_and_identical_tokens_are_unbudgeted():
    cfg, H, L = tiny_inputs()
    for mode in (orc.FROM_ALL, orc.FROM_UNION):
        for pol in (orc.SUBSTITUTION, orc.TRUNCATION):
            one = run(cfg, H[5:6], L, cfg.k, pol, mode)           # M = 1, B = k
            full = run(cfg, H[5:6], L, cfg.n_experts, pol, mode)
            assert sorted(one["S"]) == sorted(one["topk"][0])
            np.testing.assert_array_equal(one["out"], full["out"])
            same = np.repeat(H[5:6], 4, axis=0)
            rs = run(cfg, same, L, cfg.k, pol, mode)
            assert all(sorted(a) == sorted(full["assign"][0]) for a in rs["assign"])
            np.testing.assert_allclose(rs["out"], np.repeat(full["out"], 4, axis=0), rtol=0,
                                       atol=1e-13 * np.abs(full["out"]).max())   # BLAS blocks 4 rows differently from 1


def test_single_expert_is_a_plain_swiglu_ffn():
    rng = np.random.default_rng(5)
    d, f, M = 6, 10, 4                                           # f != d: a transposed operand cannot pass
    H = rng.standard_normal((M, d)); W1 = rng.standard_normal((1, f, d)); W3 = rng.standard_normal((1, f, d))
    W2 = rng.standard_normal((1, d, f)); Wr = rng.standard_normal((1, d))
    r = orc.verify_layer(H, Wr, None, W1, W3, W2, 1, 1, orc.SUBSTITUTION, orc.FROM_ALL, True)
    Ht = torch.from_numpy(H)
    ref = (torch.nn.functional.silu(Ht @ torch.from_numpy(W1[0]).T) * (Ht @ torch.from_numpy(W3[0]).T)) @ torch.from_numpy(W2[0]).T
    np.testing.assert_allclose(r["out"], ref.numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_array_equal(r["wgt"], np.ones((M, 1)))


def test_k_equals_n_is_dense_softmax_mixture():
    cfg, H, L = tiny_inputs(M=5)
    N = cfg.n_experts
    r = run(cfg, H, L, N, k=N)
    ys = np.stack([orc.expert_ffn(H, L["w_gate"][i], L["w_up"][i], L["w_down"][i]) for i in range(N)], axis=1)
    g = torch.softmax(torch.from_numpy(r["logits"]).double(), dim=1).numpy()
    ref = np.einsum("tn,tnd->td", g, ys)
    np.testing.assert_allclose(r["out"], ref, rtol=1e-11, atol=1e-13 * np.abs(ref).max())


def test_truncation_empty_intersection_gives_exact_zero_row():
    cfg, H, L = tiny_inputs()
    hit = False
    for B in (1, 2, 3):
        r = run(cfg, H, L, B, orc.TRUNCATION)
        for t in range(H.shape[0]):
            if not (set(r["topk"][t]) & set(r["S"])):
                hit = True
                assert r["assign"][t] == []
                assert not r["out"][t].any() and not r["wgt"][t].any()
    assert hit, "fixture should contain a token with no kept expert"


def test_token_permutation_equivariance():
    cfg, H, L = tiny_inputs()
    perm = np.random.default_rng(6).permutation(H.shape[0])
    a = run(cfg, H, L, 6)
    b = run(cfg, H[perm], L, 6)
    assert sorted(a["S"]) == sorted(b["S"])
    np.testing.assert_allclose(b["out"], a["out"][perm], rtol=0, atol=1e-13 * np.abs(a["out"]).max())
    assert [b["assign"][j] for j in range(len(perm))] == [a["assign"][perm[j]] for j in range(len(perm))]


def test_budget_below_k_and_logits_override():
    cfg, H, L = tiny_inputs()
    r = run(cfg, H, L, 2)                                         # B < k: min(k, |S|) experts per token
    assert all(len(a) == 2 for a in r["assign"])
    z = r["logits"].copy()
    r2 = run(cfg, H, L, 2, logits=z)
    np.testing.assert_array_equal(r2["out"], r["out"])


# ------------------------------------------------------------ O9 permutation
def test_canonical_permutation_properties():
    cfg, H, L = tiny_inputs()
    for pol in (orc.SUBSTITUTION, orc.TRUNCATION):
        r = run(cfg, H, L, 5, pol)
        A, N = r["assign"], cfg.n_experts
        R = sum(len(a) for a in A)
        assert sum(r["count"]) == R == len(r["perm_row2tok"])
        if pol == orc.SUBSTITUTION:
            assert R == H.shape[0] * min(cfg.k, len(r["S"]))
        assert r["offset"][0] == 0 and r["offset"][N] == R
        assert all(r["offset"][i + 1] - r["offset"][i] == r["count"][i] for i in range(N))
        assert r["active"] == [i for i in range(N) if r["count"][i] > 0]
        pairs = {(t, i) for t in range(len(A)) for i in A[t]}
        assert set(r["row_of"].keys()) == pairs
        assert sorted(r["row_of"].values()) == list(range(R))      # bijection onto rows
        for (t, i), row in r["row_of"].items():
            assert r["offset"][i] <= row < r["offset"][i + 1] and r["perm_row2tok"][row] == t
        for i in range(N):
            seg = r["perm_row2tok"][r["offset"][i]:r["offset"][i + 1]]
            assert seg == sorted(seg)


# ------------------------------------------------------------ storage rounding
def test_round_bf16_matches_torch():
    x = np.random.default_rng(7).standard_normal(4096) * 10
    x[:4] = [0.0, 1.00390625, 1.01171875, -3.0e-39]               # ties to even both ways, a denormal
    ref = torch.from_numpy(x.astype(np.float32)).to(torch.bfloat16).double().numpy()
    np.testing.assert_array_equal(orc.round_bf16(x), ref)


# ------------------------------------------------------------ O10 static ranking (Eq. 4)
def test_static_counts_brute_force_and_ranking():
    rng = np.random.default_rng(8)
    z = rng.integers(-3, 4, size=(57, 9)).astype(np.float32)        # ties included
    k = 3
    c = orc.static_counts(z, k)
    # brute force: expert i is in T_k(h) iff fewer than k experts rank strictly before it
    want = [0] * 9
    for t in range(z.shape[0]):
        for i in range(9):
            if sum(beats(z[t], j, i) for j in range(9)) < k:
                want[i] += 1
    assert c == want and sum(c) == z.shape[0] * k
    rank = orc.static_ranking(c)
    assert sorted(rank) == list(range(9))
    assert all(c[a] > c[b] or (c[a] == c[b] and a < b) for a, b in zip(rank, rank[1:]))
    # counts do not depend on the order of the calibration tokens, and add over calibration chunks
    perm = rng.permutation(z.shape[0])
    assert orc.static_counts(z[perm], k) == c
    c2 = [a + b for a, b in zip(orc.static_counts(z[:20], k), orc.static_counts(z[20:], k))]
    assert c2 == c


def test_static_shortlist_is_the_prefix_of_the_fixed_ordering():
    cfg, H, L = tiny_inputs()
    z = orc.router_logits(H, L["router_w"], L["router_bias"])
    rank = orc.static_ranking(orc.static_counts(z, cfg.k))
    for B in (1, 4, 8, 16, 30):
        for pol in (orc.SUBSTITUTION, orc.TRUNCATION):
            r = orc.route(z, cfg.k, B, pol, orc.STATIC, True, static_rank=rank)
            assert r["S"] == rank[:min(B, cfg.n_experts)]
            S = set(r["S"])
            for t in range(H.shape[0]):
                Tk = set(r["topk"][t])
                if pol == orc.TRUNCATION:
                    assert set(r["assign"][t]) == Tk & S
                else:
                    assert set(r["assign"][t]) <= S and len(r["assign"][t]) == min(cfg.k, len(S))
    # a budget of all N experts reproduces the unbudgeted layer whatever the ordering
    full = run(cfg, H, L, cfg.n_experts)
    st = orc.verify_layer(H, L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], cfg.k,
                          cfg.n_experts, orc.SUBSTITUTION, orc.STATIC, True, static_rank=rank)
    np.testing.assert_array_equal(st["out"], full["out"])

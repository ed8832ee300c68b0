"""Pins for the oracle's stack (O11), greedy oracle ranking (O12, Eq. 6) and reconstruction error (O13).

As in test_oracle_pins.py nothing here retypes the oracle's own formulas: a hand-worked example, brute
force, closed forms and reductions to other, separately pinned routines (the truncation layer of Eq. 7, a
plain residual SwiGLU stack written with torch).  No GPU needed.
"""
import itertools
import json
import os

import numpy as np
import pytest
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden", "handworked_greedy.json")


def layer_f64(cfg, seed, layer=0):
    L = synth.gen_layer(cfg, seed, layer)
    return {k: v.double().numpy() for k, v in L.items()}


def small_cfg(**kw):
    base = dict(d=64, n_experts=8, k=2, f=64, dtype="bf16", slope=1.0)
    base.update(kw)
    return synth.LayerConfig("small", **base)


# ------------------------------------------------------------------ O11: stack
def test_stack_with_zero_down_projection_is_the_identity():
    cfg = small_cfg()
    layers = [layer_f64(cfg, 5, l) for l in range(3)]
    for L in layers:
        L["w_down"] = np.zeros_like(L["w_down"])
    H = synth.gen_hidden(cfg, 9, 5).double().numpy()
    xs, routes = orc.verify_stack(H, layers, cfg.k, [3, 4, 5], orc.SUBSTITUTION, orc.FROM_ALL, True, "bf16")
    assert len(xs) == 4 and len(routes) == 3
    for x in xs:
        np.testing.assert_array_equal(x, H)
    assert [len(r["S"]) for r in routes] == [3, 4, 5]       # every layer uses its own budget


def test_single_expert_stack_is_a_plain_residual_swiglu_stack():
    # N = 1, k = 1: the gate weight is exactly 1, so every layer is x + W2 (silu(W1 x) * W3 x)
    cfg = small_cfg(n_experts=1, k=1)
    layers = [layer_f64(cfg, 11, l) for l in range(4)]
    H = synth.gen_hidden(cfg, 7, 11).double().numpy()
    xs, _ = orc.verify_stack(H, layers, 1, [1] * 4, orc.SUBSTITUTION, orc.FROM_ALL, True, "bf16")
    x = torch.from_numpy(H)
    for l, L in enumerate(layers):
        w1, w3, w2 = (torch.from_numpy(L[n][0]) for n in ("w_gate", "w_up", "w_down"))
        y = (torch.nn.functional.silu(x @ w1.T) * (x @ w3.T)) @ w2.T
        x = (x + y).to(torch.float32).to(torch.bfloat16).double()
        np.testing.assert_allclose(xs[l + 1], x.numpy(), rtol=0, atol=1e-12)
        # the stream holds storage values only
        assert torch.equal(x, x.to(torch.bfloat16).double())


def test_stack_layers_see_the_previous_layers_output():
    # layer l of the stack must equal a stand-alone layer call on x_l (and not on x_0)
    cfg = small_cfg()
    layers = [layer_f64(cfg, 21, l) for l in range(3)]
    H = synth.gen_hidden(cfg, 12, 21).double().numpy()
    budgets = [4, 2, 6]
    xs, routes = orc.verify_stack(H, layers, cfg.k, budgets, orc.TRUNCATION, orc.FROM_UNION, False, "fp32")
    for l, L in enumerate(layers):
        r = orc.verify_layer(xs[l], L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], cfg.k,
                             budgets[l], orc.TRUNCATION, orc.FROM_UNION, False)
        assert r["S"] == routes[l]["S"]
        np.testing.assert_array_equal(xs[l + 1], (xs[l] + r["out"]).astype(np.float32).astype(np.float64))
    assert not np.array_equal(xs[1], xs[0])


def test_round_storage_fp16_matches_torch():
    x = np.random.default_rng(3).standard_normal(4096) * np.logspace(-6, 4, 4096)
    ref = torch.from_numpy(x).to(torch.float16).double().numpy()
    np.testing.assert_array_equal(orc.round_storage(x, "fp16"), ref)


# ------------------------------------------------------------- O12: Eq. 6 greedy
def test_handworked_greedy_example():
    g = json.load(open(GOLD))
    T = g["topk"]
    C = [{int(i): np.array(v) for i, v in row.items()} for row in g["contributions"]]
    O_star = orc.gold_output(T, C, g["d"])
    np.testing.assert_array_equal(O_star, np.array(g["gold"]))
    for key, val in g["objective"].items():
        S = [int(x) for x in key.split(",")] if key else []
        assert orc.subset_error(T, C, O_star, S) == val
    order, errs = orc.oracle_ranking(T, C, g["n_experts"], g["d"], 3)
    assert order == g["order"] and errs == g["errors"]


def greedy_case(seed=2, M=10, renorm=True, **kw):
    cfg = small_cfg(**kw)
    L = layer_f64(cfg, seed)
    H = synth.gen_hidden(cfg, M, seed).double().numpy()
    z = orc.router_logits(H, L["router_w"], L["router_bias"])
    T, C = orc.expert_contributions(H, z, cfg.k, renorm, L["w_gate"], L["w_up"], L["w_down"])
    return cfg, L, H, z, T, C


@pytest.mark.parametrize("renorm", [True, False])
def test_gold_output_is_the_unbudgeted_layer(renorm):
    cfg, L, H, z, T, C = greedy_case(renorm=renorm)
    full = orc.verify_layer(H, L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], cfg.k,
                            cfg.n_experts, orc.SUBSTITUTION, orc.FROM_ALL, renorm)
    np.testing.assert_allclose(orc.gold_output(T, C, cfg.d), full["out"], rtol=0, atol=1e-13)


@pytest.mark.parametrize("renorm", [True, False])
def test_subset_objective_is_the_truncation_layers_error(renorm):
    # for a fixed shortlist S the inner sum of Eq. 6 is the truncation output of Eq. 7 (weights over the
    # original top-k), which is pinned on its own; checked for every subset of size <= 2 and a few larger
    cfg, L, H, z, T, C = greedy_case(renorm=renorm)
    O_star = orc.gold_output(T, C, cfg.d)
    N = cfg.n_experts
    subsets = [list(c) for r in (0, 1, 2) for c in itertools.combinations(range(N), r)] + [[0, 3, 5, 6], list(range(N))]
    for S in subsets:
        if S:
            r = orc.verify_layer(H, L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], cfg.k,
                                 len(S), orc.TRUNCATION, orc.STATIC, renorm, static_rank=S)
            want = float(np.sum((O_star - r["out"]) ** 2))
        else:
            want = float(np.sum(O_star ** 2))
        assert orc.subset_error(T, C, O_star, S) == pytest.approx(want, rel=1e-10, abs=1e-22)


def test_greedy_steps_are_brute_force_minimisers_and_errors_decrease_to_zero():
    cfg, L, H, z, T, C = greedy_case(seed=4, M=12)
    N = cfg.n_experts
    O_star = orc.gold_output(T, C, cfg.d)
    order, errs = orc.oracle_ranking(T, C, N, cfg.d, N)
    assert sorted(order) == list(range(N))
    for b in range(N):
        cands = {i: orc.subset_error(T, C, O_star, order[:b] + [i]) for i in range(N) if i not in order[:b]}
        best = min(cands.values())
        assert errs[b] == best
        assert order[b] == min(i for i, e in cands.items() if e == best)
    # first pick: the best single expert over all N (brute force), and shorter budgets are prefixes
    assert orc.oracle_ranking(T, C, N, cfg.d, 3)[0] == order[:3]
    union = sorted({i for row in T for i in row})
    n_needed = max(order.index(i) for i in union) + 1
    assert errs[n_needed - 1] <= 1e-25 * max(1.0, float(np.sum(O_star ** 2)))
    # the first pick can always fall back on an expert without rows, so it never exceeds the empty set's objective
    assert errs[0] <= float(np.sum(O_star ** 2)) + 1e-12


def test_greedy_with_k1_sorts_experts_by_their_output_energy():
    # k = 1: every token has one term, tokens do not interact, so the objective after picking S is the
    # total energy minus the energy of the picked experts' tokens: greedy = sort by energy, descending
    cfg, L, H, z, T, C = greedy_case(seed=6, M=14, k=1)
    N = cfg.n_experts
    energy = [sum(float(C[t][i] @ C[t][i]) for t in range(len(T)) if i in T[t]) for i in range(N)]
    want = sorted(range(N), key=lambda i: (-energy[i], i))
    order, errs = orc.oracle_ranking(T, C, N, cfg.d, N)
    assert order == want
    total = sum(energy)
    run = 0.0
    for b, i in enumerate(order):
        run += energy[i]
        assert errs[b] == pytest.approx(total - run, rel=1e-9, abs=1e-20)


# ------------------------------------------------- O13: reconstruction error
def test_reconstruction_error_closed_forms():
    rng = np.random.default_rng(0)
    O = rng.standard_normal((5, 16))
    assert orc.reconstruction_error(O, O) == 0.0
    assert orc.reconstruction_error(np.zeros_like(O), O) == pytest.approx(1.0, rel=1e-15)
    assert orc.reconstruction_error(1.25 * O, O) == pytest.approx(0.0625, rel=1e-12)
    assert orc.reconstruction_error(-O, O) == pytest.approx(4.0, rel=1e-12)
    D = rng.standard_normal(O.shape)
    e1 = orc.reconstruction_error(O + D, O)
    assert orc.reconstruction_error(3.0 * (O + D), 3.0 * O) == pytest.approx(e1, rel=1e-12)   # scale invariant
    assert e1 == pytest.approx(np.linalg.norm(D) ** 2 / np.linalg.norm(O) ** 2, rel=1e-12)


def test_greedy_error_curve_is_the_reconstruction_error_of_the_truncation_layer():
    cfg, L, H, z, T, C = greedy_case(seed=8, M=10)
    O_star = orc.gold_output(T, C, cfg.d)
    order, errs = orc.oracle_ranking(T, C, cfg.n_experts, cfg.d, 5)
    den = float(np.sum(O_star ** 2))
    for b in range(5):
        r = orc.verify_layer(H, L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], cfg.k, b + 1,
                             orc.TRUNCATION, orc.STATIC, True, static_rank=order)
        assert orc.reconstruction_error(r["out"], O_star) == pytest.approx(errs[b] / den, rel=1e-9, abs=1e-20)
    # and greedy is at least as good as the router-based shortlist of the same size on its own objective
    # at B = 1 (it is the brute-force optimum there)
    rb = orc.route(z, cfg.k, 1, orc.TRUNCATION, orc.FROM_ALL, True)["S"]
    assert errs[0] <= orc.subset_error(T, C, O_star, rb) + 1e-15

"""Analysis mode on the GPU against the CPU oracle: oracle ranking (Eq. 6) and reconstruction error (Section 4.5).

The greedy loop takes an argmin over floating-point objectives, so it is checked in two ways.  (1) In the
same precision: the oracle is given the GPU's own expert rows (fp32 accumulators times the fp32 mixing
weights), after which the Gram matrices must agree to rounding and every pick must be the oracle's
minimiser.  (2) End to end against the fp64 oracle (fp64 FFNs): at every step, with the GPU's earlier
picks as the state, the GPU's pick must be the oracle's minimiser whenever the runner-up is clearly worse,
and within tolerance of the minimum otherwise (both are then valid greedy choices).
"""
import numpy as np
import pytest
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu


def ms():
    from paper_2602_16052_b200 import moespec
    return moespec


def make_layer(case, max_M, max_k, **kw):
    return ms().Layer(case["router_w"], case["router_bias"], case["w_gate"], case["w_up"], case["w_down"],
                      max_M=max_M, max_k=max_k, **kw)


def gpu_contributions(layer, M, k):
    """C[t][i] from what the unpruned GPU pass left behind: y rows (fp32) times mixing weights (fp32)."""
    g = layer.get_routing()
    y = layer.get_intermediate("y", g["n_rows"]).double().numpy()
    T = [[int(e) for e in g["assign_idx"][t] if e >= 0] for t in range(M)]
    C = [dict() for _ in range(M)]
    for t in range(M):
        for a in range(k):
            e, row = int(g["assign_idx"][t, a]), int(g["tokslot2row"][t, a])
            if e >= 0:
                C[t][e] = float(g["gate_w"][t, a]) * y[row]
    return T, C, g


def candidates_objective(T, C, O_star, S, N):
    return {i: orc.subset_error(T, C, O_star, list(S) + [i]) for i in range(N) if i not in S}


@pytest.mark.parametrize("renorm,M,n_pick", [(True, 63, 24), (False, 31, 64), (True, 1, 10)])
def test_oracle_ranking_in_the_gpus_own_precision(renorm, M, n_pick):
    cfg = synth.CONFIGS["olmoe"].with_(f=256)
    case = H.make_case(cfg, M, seed=61)
    layer = make_layer(case, 64, cfg.k, renormalize=renorm, policy=ms().TRUNCATION, shortlist=ms().FROM_UNION,
                       out_dtype=torch.float32)             # the analysis ignores policy and shortlist mode
    out_star = torch.empty((M, cfg.d), dtype=torch.float32, device="cuda")
    order, obj, gold = layer.oracle_ranking(case["hidden"], cfg.k, n_pick, out_star)
    assert len(set(order)) == n_pick and all(0 <= e < cfg.n_experts for e in order)
    T, C, g = gpu_contributions(layer, M, cfg.k)
    assert layer.get_stats()["n_active"] == len({e for row in T for e in row})      # the unpruned pass

    # Gram matrices: G[t][a][b] = c_{t,a} . c_{t,b}
    G = layer.get_gram()
    for t in range(M):
        rows = np.stack([C[t][int(g["assign_idx"][t, a])] for a in range(cfg.k)])
        want = rows @ rows.T
        np.testing.assert_allclose(G[t], want, rtol=1e-11, atol=1e-13 * float(np.abs(want).max()))

    # O* written by the pass is the sum of the contributions (fp32 combine)
    O_star = orc.gold_output(T, C, cfg.d)
    np.testing.assert_allclose(out_star.double().cpu().numpy(), O_star, rtol=0,
                               atol=4e-6 * float(np.abs(O_star).max()))
    total = float(np.sum(O_star ** 2))
    assert gold == pytest.approx(total, rel=1e-10)

    # every pick is the minimiser of the objective evaluated from its definition
    S = []
    for b, pick in enumerate(order):
        cand = candidates_objective(T, C, O_star, S, cfg.n_experts)
        best = min(cand.values())
        near = [i for i, e in cand.items() if e - best <= 1e-9 * total]
        assert pick in near, f"step {b}: picked {pick}, minimisers {near}"
        if len(near) == 1 or all(cand[i] == best for i in near):
            assert pick == min(near)                      # unique minimiser, or exact tie -> lower index
        assert obj[b] == pytest.approx(cand[pick], rel=0, abs=1e-9 * total)
        S.append(pick)
    if n_pick == cfg.n_experts:
        assert abs(obj[-1]) <= 1e-9 * total
    layer.destroy()


def test_oracle_ranking_against_the_fp64_oracle():
    cfg = synth.CONFIGS["olmoe"].with_(f=256)
    M, n_pick = 63, 32
    case = H.make_case(cfg, M, seed=62)
    layer = make_layer(case, M, cfg.k, out_dtype=torch.float32)
    order, obj, gold = layer.oracle_ranking(case["hidden"], cfg.k, n_pick)
    z = layer.get_logits()
    T, C = orc.expert_contributions(H.f64(case["hidden"]), z, cfg.k, True, H.LazyF64(case["w_gate"]),
                                    H.LazyF64(case["w_up"]), H.LazyF64(case["w_down"]))
    O_star = orc.gold_output(T, C, cfg.d)
    total = float(np.sum(O_star ** 2))
    assert gold == pytest.approx(total, rel=2e-2)
    S, decisive = [], 0
    prev = total
    for b, pick in enumerate(order):
        cand = candidates_objective(T, C, O_star, S, cfg.n_experts)
        ranked = sorted(cand.items(), key=lambda kv: (kv[1], kv[0]))
        best_i, best = ranked[0]
        gain = prev - best
        tol = 0.05 * abs(gain) + 1e-3 * total / cfg.n_experts
        assert cand[pick] - best <= tol, f"step {b}: pick {pick} is {cand[pick] - best:.3e} above the minimum"
        if ranked[1][1] - best > tol:
            decisive += 1
            assert pick == best_i, f"step {b}: clear minimiser {best_i}, GPU picked {pick}"
        assert obj[b] == pytest.approx(cand[pick], rel=0, abs=2e-2 * total)
        S.append(pick)
        prev = cand[pick]
    assert decisive >= n_pick // 2, "the fixture should have mostly clear-cut steps"
    # the method's point (Section 4.5): at equal size the greedy set reconstructs at least as well as the
    # router-based shortlist, on the oracle's own numbers
    r = orc.route(z, cfg.k, n_pick, orc.TRUNCATION, orc.FROM_ALL, True)
    assert orc.subset_error(T, C, O_star, order) <= orc.subset_error(T, C, O_star, r["S"]) * (1 + 1e-2)
    layer.destroy()


def test_reconstruction_error_of_router_static_and_oracle_shortlists():
    """||O_S - O*||^2 / ||O*||^2 on the GPU for the three ranking strategies of Section 3.2, each against the
    oracle's value for the same shortlist; and the reduction itself against closed forms."""
    m = ms()
    cfg = synth.CONFIGS["olmoe"].with_(f=256)
    M, B = 63, 16
    case = H.make_case(cfg, M, seed=63)
    hidden = case["hidden"]
    full = make_layer(case, M, cfg.k, out_dtype=torch.float32)
    O_star = torch.empty((M, cfg.d), dtype=torch.float32, device="cuda")
    order, obj, gold = full.oracle_ranking(hidden, cfg.k, B, O_star)
    z = full.get_logits()

    # closed forms of the reduction
    assert full.reconstruction_error(O_star, O_star)[0] == 0.0
    assert full.reconstruction_error(torch.zeros_like(O_star), O_star)[0] == pytest.approx(1.0, rel=1e-12)
    err, num, den = full.reconstruction_error(1.25 * O_star, O_star)
    assert err == pytest.approx(0.0625, rel=1e-6) and den == pytest.approx(gold, rel=1e-5)
    noisy = O_star + 0.1 * torch.randn_like(O_star)
    want = orc.reconstruction_error(noisy.double().cpu().numpy(), O_star.double().cpu().numpy())
    assert full.reconstruction_error(noisy, O_star)[0] == pytest.approx(want, rel=1e-12)

    # fp64 reference for O*
    ref_full = H.oracle_run(case, cfg.k, cfg.n_experts, orc.SUBSTITUTION, orc.FROM_ALL, True, logits=z)
    errs = {}
    for name, mode, omode, rank in (("router", m.FROM_ALL, orc.FROM_ALL, None), ("oracle", m.STATIC, orc.STATIC, order)):
        lay = make_layer(case, M, cfg.k, policy=m.TRUNCATION, shortlist=mode, out_dtype=torch.float32)
        if rank is not None:
            lay.set_static_ranking(rank)
        O_S = lay.verify_layer(hidden, cfg.k, B)
        got = full.reconstruction_error(O_S, O_star)[0]
        r = H.oracle_run(case, cfg.k, B, orc.TRUNCATION, omode, True, logits=lay.get_logits(), static_rank=rank)
        want = orc.reconstruction_error(r["out"], ref_full["out"])
        assert got == pytest.approx(want, rel=3e-2, abs=1e-4), name
        errs[name] = got
        lay.destroy()
    # the oracle's objective after B picks is the same quantity (truncation output of its shortlist)
    assert errs["oracle"] == pytest.approx(obj[B - 1] / gold, rel=1e-3, abs=1e-6)
    assert errs["oracle"] <= errs["router"] * (1 + 1e-2)
    full.destroy()


def test_analysis_argument_errors():
    m = ms()
    cfg = synth.CONFIGS["olmoe"].with_(f=128, n_experts=16)
    case = H.make_case(cfg, 8, seed=64)
    layer = make_layer(case, 8, cfg.k, out_dtype=torch.float32)
    with pytest.raises(m.MoeSpecError):
        layer.get_gram()                                      # nothing computed yet
    for bad in (0, cfg.n_experts + 1):
        with pytest.raises(m.MoeSpecError) as ei:
            layer.oracle_ranking(case["hidden"], cfg.k, bad)
        assert ei.value.code == m.ERR_INVALID_ARG
    with pytest.raises(m.MoeSpecError):
        layer.oracle_ranking(torch.cat([case["hidden"], case["hidden"]]), cfg.k, 4)    # M > max_M
    order, obj, gold = layer.oracle_ranking(case["hidden"], cfg.k, cfg.n_experts)
    assert sorted(order) == list(range(cfg.n_experts)) and abs(obj[-1]) <= 1e-9 * gold
    layer.destroy()

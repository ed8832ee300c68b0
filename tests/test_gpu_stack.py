"""The residual stack entry point (L layers, one graph launch, per-layer budgets) against the CPU oracle.

Routing decisions are discrete, so a free-running comparison over many layers would measure how often a
near-tie flips, not the arithmetic.  Every layer is therefore checked on its own: the oracle runs layer l on
the GPU stack's x_l (read back through moespec_stack_get_stream) and the result must match x_{l+1} within
the single-layer bar plus the rounding of the stored stream.
"""
import numpy as np
import pytest
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import synth
from tests import helpers as H

pytestmark = pytest.mark.gpu

BF16_TOL = 2e-2


def ms():
    from paper_2602_16052_b200 import moespec
    return moespec


def build_stack(cfg, max_M, seed, **kw):
    m = ms()
    cases = [synth.gen_layer(cfg, seed, l, "cuda") for l in range(cfg.n_layers)]
    layers = [m.Layer(c["router_w"], c["router_bias"], c["w_gate"], c["w_up"], c["w_down"], max_M=max_M,
                      max_k=cfg.k, residual=True, **kw) for c in cases]
    return cases, layers, m.Stack(layers)


def check_layers(cfg, cases, layers, xs, budgets, policy, mode, renorm):
    for l, (case, layer) in enumerate(zip(cases, layers)):
        x_l = H.f64(xs[l])
        c = dict(case)
        c["hidden"] = xs[l]
        z_gpu = layer.get_logits()
        z_ref = orc.router_logits(x_l, H.f64(case["router_w"]), H.f64(case["router_bias"]))
        assert np.max(np.abs(z_gpu.astype(np.float64) - z_ref)) <= 2e-5 * max(1.0, np.abs(z_ref).max()), f"logits of layer {l}"
        r = H.oracle_run(c, cfg.k, budgets[l], policy, mode, renorm, logits=z_gpu)
        H.compare_routing(layer.get_routing(), r, policy, cfg.k)
        assert layer.get_stats()["status"] == 0
        nxt = x_l + r["out"]
        rms = float(np.sqrt(np.mean(r["out"] ** 2)))
        bound = BF16_TOL * rms + 2.0 ** -8 * np.abs(nxt)
        got = H.f64(xs[l + 1])
        assert np.all(np.abs(got - nxt) <= bound), f"layer {l}: worst {np.max(np.abs(got - nxt) / bound):.2f}x of bound"


@pytest.mark.parametrize("policy_name,mode_name,renorm", [("SUBSTITUTION", "FROM_ALL", True),
                                                           ("TRUNCATION", "FROM_UNION", False)])
def test_stack_per_layer_parity_with_per_layer_budgets(policy_name, mode_name, renorm):
    m = ms()
    cfg = synth.CONFIGS["olmoe"].with_(f=256, n_experts=32, n_layers=5)
    M = 37
    budgets = [12, 6, 20, 32, 9]
    policy, mode = getattr(m, policy_name), getattr(m, mode_name)
    cases, layers, stack = build_stack(cfg, M, seed=31, policy=policy, shortlist=mode, renormalize=renorm)
    x0 = synth.gen_hidden(cfg, M, seed=31, device="cuda")
    out = stack.verify_stack(x0, cfg.k, budgets)
    torch.cuda.synchronize()
    assert stack.last_launch_count() == 4 * cfg.n_layers
    xs = [x0.cpu()] + [stack.get_stream(l) for l in range(1, cfg.n_layers)] + [out.cpu()]
    check_layers(cfg, cases, layers, xs, budgets, getattr(orc, policy_name), getattr(orc, mode_name), renorm)
    for l, layer in enumerate(layers):
        assert layer.get_stats()["n_shortlist"] <= budgets[l]

    # replays of the cached graph, the kernel-by-kernel path and layer-by-layer calls give the same bits
    again = stack.verify_stack(x0, cfg.k, budgets).clone()
    stack.set_graph(False)
    plain = stack.verify_stack(x0, cfg.k, budgets).clone()
    stack.set_graph(True)
    cur = x0
    for l, layer in enumerate(layers):
        cur = layer.verify_layer(cur, cfg.k, budgets[l]).clone()
    torch.cuda.synchronize()
    assert torch.equal(out, again) and torch.equal(out, plain) and torch.equal(out, cur)

    # new budgets and a new tree size re-capture; the result follows the arguments, not the cache
    b2 = [8] * cfg.n_layers
    M2 = 19
    out2 = stack.verify_stack(x0[:M2].contiguous(), cfg.k, b2)
    torch.cuda.synchronize()
    xs2 = [x0[:M2].cpu()] + [stack.get_stream(l) for l in range(1, cfg.n_layers)] + [out2.cpu()]
    assert xs2[1].shape[0] == M2
    check_layers(cfg, cases, layers, xs2, b2, getattr(orc, policy_name), getattr(orc, mode_name), renorm)
    stack.destroy()
    for layer in layers:
        layer.destroy()


def test_stack_at_full_layer_size():
    """All 16 layers of the benchmark stack at their full size (d=2048, N=64, f=1024, M=63, B=32), in the
    configuration the benchmark times (one graph launch, bf16 residual stream), each layer checked against
    the oracle on the GPU's own input to that layer."""
    cfg = synth.CONFIGS["olmoe16"]
    M, B = 63, 32
    cases, layers, stack = build_stack(cfg, M, seed=2000)
    x0 = synth.gen_hidden(cfg, M, seed=2000, device="cuda")
    out = stack.verify_stack(x0, cfg.k, B)
    torch.cuda.synchronize()
    xs = [x0.cpu()] + [stack.get_stream(l) for l in range(1, cfg.n_layers)] + [out.cpu()]
    check_layers(cfg, cases, layers, xs, [B] * cfg.n_layers, orc.SUBSTITUTION, orc.FROM_ALL, True)
    for layer in layers:
        assert layer.get_stats()["n_active"] == B
    stack.destroy()
    for layer in layers:
        layer.destroy()


def test_wide_router_stack_at_full_layer_size():
    """Three layers of the 48-layer Qwen3-30B-A3B-shaped stack at full size (d=2048, N=128, k=8, f=768),
    renormalised gating and one graph launch per pass as the benchmark tables run it, at all six points of its
    (M, B) sweep; each layer checked against the oracle on the GPU's own input to that layer."""
    cfg = synth.CONFIGS["qwen3"].with_(n_layers=3)
    cases, layers, stack = build_stack(cfg, 127, seed=2000)
    for M, B in ((63, 32), (63, 64), (63, 128), (127, 32), (127, 64), (127, 128)):
        x0 = synth.gen_hidden(cfg, M, seed=2000, device="cuda")
        out = stack.verify_stack(x0, cfg.k, B)
        torch.cuda.synchronize()
        xs = [x0.cpu()] + [stack.get_stream(l) for l in range(1, cfg.n_layers)] + [out.cpu()]
        check_layers(cfg, cases, layers, xs, [B] * cfg.n_layers, orc.SUBSTITUTION, orc.FROM_ALL, True)
    stack.destroy()
    for layer in layers:
        layer.destroy()


def test_stack_host_entry_and_static_ranking_change():
    m = ms()
    cfg = synth.CONFIGS["olmoe"].with_(f=128, n_experts=16, n_layers=3)
    M, budgets = 21, [6, 6, 6]
    cases, layers, stack = build_stack(cfg, M, seed=41, shortlist=m.STATIC)
    x0 = synth.gen_hidden(cfg, M, seed=41, device="cuda")
    with pytest.raises(m.MoeSpecError):            # STATIC layers without a ranking are refused
        stack.verify_stack(x0, cfg.k, budgets)
    order_a = list(range(cfg.n_experts))
    order_b = order_a[::-1]
    for layer in layers:
        layer.set_static_ranking(order_a)
    out_a = stack.verify_stack(x0, cfg.k, budgets).clone()
    h_in = x0.cpu().pin_memory()
    h_out = torch.empty_like(h_in).pin_memory()
    stack.verify_stack_host(h_in, cfg.k, budgets, h_out)
    assert torch.equal(h_out, out_a.cpu())
    pageable = torch.empty_like(x0, device="cpu")
    stack.verify_stack_host(x0.cpu(), cfg.k, budgets, pageable)
    assert torch.equal(pageable, out_a.cpu())
    # a new ranking must invalidate the cached graph (its size is a kernel argument)
    for layer in layers:
        layer.set_static_ranking(order_b[:8])
    out_b = stack.verify_stack(x0, cfg.k, budgets).clone()
    torch.cuda.synchronize()
    assert not torch.equal(out_a, out_b)
    xs = [x0.cpu()] + [stack.get_stream(l) for l in range(1, cfg.n_layers)] + [out_b.cpu()]
    for l, (case, layer) in enumerate(zip(cases, layers)):
        c = dict(case)
        c["hidden"] = xs[l]
        r = H.oracle_run(c, cfg.k, budgets[l], orc.SUBSTITUTION, orc.STATIC, True, logits=layer.get_logits(),
                         static_rank=order_b[:8])
        assert layer.get_routing()["S"] == r["S"] == order_b[:6]
        nxt = H.f64(xs[l]) + r["out"]
        bound = BF16_TOL * float(np.sqrt(np.mean(r["out"] ** 2))) + 2.0 ** -8 * np.abs(nxt)
        assert np.all(np.abs(H.f64(xs[l + 1]) - nxt) <= bound)
    stack.destroy()
    for layer in layers:
        layer.destroy()


def test_stack_argument_errors():
    m = ms()
    cfg = synth.CONFIGS["olmoe"].with_(f=128, n_experts=16, n_layers=2)
    cases = [synth.gen_layer(cfg, 51, l, "cuda") for l in range(2)]
    mk = lambda c, **kw: m.Layer(c["router_w"], c["router_bias"], c["w_gate"], c["w_up"], c["w_down"], max_M=16,
                                 max_k=cfg.k, **kw)
    no_res = mk(cases[0])
    fp32_out = mk(cases[1], residual=True, out_dtype=torch.float32)
    a, b = mk(cases[0], residual=True), mk(cases[1], residual=True)
    for bad in ([no_res, b], [a, fp32_out], [a, a], []):
        with pytest.raises(m.MoeSpecError) as ei:
            m.Stack(bad)
        assert ei.value.code == m.ERR_INVALID_ARG
    stack = m.Stack([a, b])
    x = synth.gen_hidden(cfg, 16, seed=51, device="cuda")
    with pytest.raises(ValueError):
        stack.verify_stack(x, cfg.k, [4])                       # one budget per layer
    with pytest.raises(m.MoeSpecError):
        stack.verify_stack(x, cfg.k, [4, 0])                    # B >= 1
    with pytest.raises(m.MoeSpecError):
        stack.verify_stack(torch.cat([x, x]), cfg.k, [4, 4])    # M > max_M
    with pytest.raises(m.MoeSpecError):
        stack.verify_stack(x, cfg.k, [4, 4], out=x)             # aliasing
    assert stack.verify_stack(x[:0], cfg.k, [4, 4]).shape[0] == 0
    b.destroy()
    with pytest.raises(m.MoeSpecError) as ei:
        stack.verify_stack(x, cfg.k, [4, 4])                    # a member layer is gone
    assert ei.value.code == m.ERR_BAD_HANDLE
    stack.destroy()
    for layer in (no_res, fp32_out, a):
        layer.destroy()

"""Expert-parallel shards against the CPU oracle, on ONE GPU: the G shards of a layer run one after the other
on the same device (each holds only its block of the experts' weights), their partial outputs are added in
rank order in fp32, and the sum must match the oracle's layer output at the usual bar.  Every shard must take
exactly the oracle's routing decisions (the router is replicated, nothing is exchanged), stream only its
resident kept experts, and return exact zeros for a token none of whose kept experts it holds."""
import numpy as np
import pytest
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import ep, synth
from tests import helpers as H
from tests.test_gpu_parity import BF16_TOL, FP32_TOL

pytestmark = pytest.mark.gpu


def ms():
    from paper_2602_16052_b200 import moespec
    return moespec


def shard_layer(case, rank, world, N, **kw):
    first, count = ep.expert_range(rank, world, N)
    sl = slice(first, first + count)
    return ms().Layer(case["router_w"], case["router_bias"], case["w_gate"][sl], case["w_up"][sl], case["w_down"][sl],
                      resident=(first, count), out_dtype=torch.float32, **kw), (first, count)


def run_sharded(cfg, M, B, world, policy, mode, renorm, ffn_kernel, seed=0):
    m = ms()
    case = H.make_case(cfg, M, seed)
    N = cfg.n_experts
    whole = m.Layer(case["router_w"], case["router_bias"], case["w_gate"], case["w_up"], case["w_down"], max_M=M,
                    max_k=cfg.k, policy=policy, shortlist=mode, renormalize=renorm, ffn_kernel=ffn_kernel,
                    out_dtype=torch.float32)
    out_whole = whole.verify_layer(case["hidden"], cfg.k, B).clone()
    z = whole.get_logits()
    r = H.oracle_run(case, cfg.k, B, policy, mode, renorm, logits=z)
    H.compare_routing(whole.get_routing(), r, policy, cfg.k)
    whole.destroy()
    Hf = H.f64(case["hidden"])
    partials, n_active = [], 0
    for rank in range(world):
        layer, (first, count) = shard_layer(case, rank, world, N, max_M=M, max_k=cfg.k, policy=policy, shortlist=mode,
                                            renormalize=renorm, ffn_kernel=ffn_kernel)
        part = layer.verify_layer(case["hidden"], cfg.k, B)
        torch.cuda.synchronize()
        st = layer.get_stats()
        assert st["status"] == 0
        assert np.array_equal(layer.get_logits(), z)             # replicated router: the same logits, bit for bit
        H.compare_routing(layer.get_routing(), r, policy, cfg.k)  # ... and the oracle's routing on every shard
        mine = [e for e in r["active"] if first <= e < first + count]
        assert st["n_active"] == len(mine) and st["weight_bytes"] == len(mine) * cfg.expert_weight_bytes()
        n_active += st["n_active"]
        # the shard's own partial sum: the oracle's outer sum with the other shards' weight columns zeroed
        Wt = r["wgt"].copy()
        Wt[:, :first] = 0.0
        Wt[:, first + count:] = 0.0
        ref = orc.layer_output(Hf, Wt, H.LazyF64(case["w_gate"]), H.LazyF64(case["w_up"]), H.LazyF64(case["w_down"]))
        o = H.f64(part)
        dead = ~np.any(Wt != 0.0, axis=1)
        assert not np.any(o[dead]), "a token without a resident kept expert must get exact zeros"
        rms = float(np.sqrt(np.mean(r["out"] ** 2)))             # scale of the LAYER output
        tol = BF16_TOL * rms if cfg.dtype == "bf16" else FP32_TOL * max(rms, float(np.abs(r["out"]).max()))
        assert np.max(np.abs(o - ref)) <= tol, f"shard {rank}/{world}"
        partials.append(part.clone())
        layer.destroy()
    assert n_active == len(r["active"])                          # every active expert was streamed exactly once
    total = ep.sum_in_rank_order(partials)
    o = H.f64(total)
    rms = float(np.sqrt(np.mean(r["out"] ** 2)))
    if cfg.dtype == "bf16":
        assert np.max(np.abs(o - r["out"])) <= BF16_TOL * rms
    else:
        assert np.all(np.abs(o - r["out"]) <= FP32_TOL * np.maximum(np.abs(r["out"]), rms))
    # and the one-GPU layer computes the same thing up to the order of the outer sum
    assert np.max(np.abs(o - H.f64(out_whole))) <= 1e-5 * max(rms, float(np.abs(r["out"]).max()))


@pytest.mark.parametrize("world", [2, 4, 8])
def test_olmoe_shards_on_one_gpu(world):
    cfg = synth.CONFIGS["olmoe"]
    run_sharded(cfg, 63, 32, world, orc.SUBSTITUTION, orc.FROM_ALL, True, ms().FFN_TENSOR_CORE)


def test_mixtral_shape_two_shards_reduced_width():
    # the model the paper ran on two GPUs (Table 3): 8 experts, 4 per GPU
    cfg = synth.CONFIGS["mixtral"].with_(f=1792)
    run_sharded(cfg, 63, 6, 2, orc.SUBSTITUTION, orc.FROM_ALL, True, ms().FFN_TENSOR_CORE)


@pytest.mark.parametrize("world,policy,mode", [(3, orc.TRUNCATION, orc.FROM_UNION), (5, orc.SUBSTITUTION, orc.FROM_ALL)])
def test_uneven_shards_large_tree_and_truncation(world, policy, mode):
    # 255 tokens (no early start: the unit list takes the large-tree path), blocks of unequal size
    cfg = synth.CONFIGS["olmoe"].with_(f=256)
    run_sharded(cfg, 255, 20, world, policy, mode, True, ms().FFN_TENSOR_CORE, seed=3)


def test_tiny_fp32_shards_cuda_core_kernel():
    cfg = synth.CONFIGS["tiny"]
    for world in (2, 4):
        run_sharded(cfg, 15, 8, world, orc.SUBSTITUTION, orc.FROM_ALL, True, ms().FFN_AUTO)
        run_sharded(cfg, 15, 3, world, orc.TRUNCATION, orc.FROM_ALL, False, ms().FFN_AUTO)


def test_shard_argument_errors():
    m = ms()
    cfg = synth.CONFIGS["tiny"]
    case = H.make_case(cfg, 15)
    mk = lambda res, **kw: m.Layer(case["router_w"], case["router_bias"], case["w_gate"][res[0]:res[0] + res[1]],
                                   case["w_up"][res[0]:res[0] + res[1]], case["w_down"][res[0]:res[0] + res[1]],
                                   max_M=15, max_k=4, resident=res, **kw)
    with pytest.raises(m.MoeSpecError) as e:
        mk((4, 4), residual=True)                                # the residual is added once, after the reduction
    assert e.value.code == m.ERR_INVALID_ARG
    lib = m.lib()
    desc_ok = mk((12, 4))
    desc_ok.destroy()
    d = m.LayerDesc(d=cfg.d, n_experts=16, f=cfg.f, max_M=15, max_k=4, dtype=m.FP32, out_dtype=0, policy=1, shortlist=1,
                    renormalize=1, residual=0, ffn_kernel=0, device=0, router_w=case["router_w"].data_ptr(),
                    router_bias=None, w_gate=case["w_gate"].data_ptr(), w_up=case["w_up"].data_ptr(),
                    w_down=case["w_down"].data_ptr(), resident_first=13, resident_count=4)
    import ctypes
    h = ctypes.c_void_p()
    assert lib.moespec_layer_create(ctypes.byref(d), ctypes.byref(h)) == m.ERR_INVALID_ARG      # 13 + 4 > 16
    d.resident_first, d.resident_count = 2, 0
    assert lib.moespec_layer_create(ctypes.byref(d), ctypes.byref(h)) == m.ERR_INVALID_ARG      # a first without a count


def test_seeded_sweep_of_sharded_layers():
    """Sixteen seeded draws of (N, k, M, B, d, f, shortlist mode, slope, number of shards) through run_sharded:
    uneven expert blocks (N not a multiple of the shard count), shards that end up without a kept expert,
    trees with and without the early start."""
    import random
    rng = random.Random(20260218)
    for trial in range(16):
        N = rng.choice([4, 8, 13, 32, 64, 100])
        k = rng.randint(1, min(N, 8))
        M = rng.choice([1, 5, 16, 17, 63, 100, 129, 200])
        B = rng.randint(1, N + 1)
        cfg = synth.LayerConfig(f"epsweep{trial}", d=rng.choice([128, 256, 512]), n_experts=N, k=k,
                                f=rng.choice([128, 256]), dtype="bf16", slope=rng.choice([0.5, 1.0, 2.0]))
        world = rng.choice([w for w in (2, 3, 4, 8) if w <= N])
        mode = rng.choice([orc.FROM_ALL, orc.FROM_UNION])
        try:
            run_sharded(cfg, M, B, world, orc.SUBSTITUTION, mode, True, ms().FFN_TENSOR_CORE, seed=400 + trial)
        except AssertionError as e:
            raise AssertionError(f"trial {trial}: N={N} k={k} M={M} B={B} d={cfg.d} f={cfg.f} shards={world} "
                                 f"mode={mode}: {e}") from e

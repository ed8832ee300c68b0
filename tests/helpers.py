"""Shared test plumbing: seeded cases, oracle runs on the CPU, comparisons.  No method arithmetic."""
import numpy as np
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import synth


class LazyF64:
    """Indexable view that converts one expert's weights to fp64 numpy on demand."""

    def __init__(self, t: torch.Tensor):
        self.t = t

    def __getitem__(self, i):
        return self.t[i].to("cpu", torch.float64).numpy()


def make_case(cfg, M, seed=0, layer=0, device="cuda"):
    L = synth.gen_layer(cfg, seed, layer, device)
    L["hidden"] = synth.gen_hidden(cfg, M, seed, layer, device)
    return L


def f64(t):
    return t.to("cpu", torch.float64).numpy()


def oracle_run(case, k, B, policy, mode, renorm, logits=None, static_rank=None):
    return orc.verify_layer(f64(case["hidden"]), f64(case["router_w"]),
                            None if case["router_bias"] is None else f64(case["router_bias"]),
                            LazyF64(case["w_gate"]), LazyF64(case["w_up"]), LazyF64(case["w_down"]),
                            k, B, policy, mode, renorm, logits=logits, static_rank=static_rank)


def oracle_route(logits, k, B, policy, mode, renorm):
    return orc.route(np.asarray(logits, dtype=np.float32), k, B, policy, mode, renorm)


def selection_margins(r, k, cand=None):
    """Smallest gaps the selection depended on: (logit gap at the k/k+1 cut over all tokens,
    score gap between the worst kept and the best rejected shortlist candidate)."""
    z = np.sort(r["logits"].astype(np.float64), axis=1)[:, ::-1]
    N = z.shape[1]
    zgap = float(np.min(z[:, k - 1] - z[:, k])) if k < N else float("inf")
    cand = list(range(N)) if cand is None else list(cand)
    kept = set(r["S"])
    out = [r["score"][j] for j in cand if j not in kept]
    sgap = float(min(r["score"][i] for i in kept) - max(out)) if out and kept else float("inf")
    return zgap, sgap


def compare_routing(g, r, policy, k):
    """Bit-exact comparison of the GPU routing state `g` with the oracle result `r`."""
    M = len(r["assign"])
    assert g["S"] == r["S"], "shortlist (rank order)"
    kk = min(k, r["logits"].shape[1])
    for t in range(M):
        assert g["topk_idx"][t, :kk].tolist() == r["topk"][t], f"natural top-k of token {t}"
        got = g["assign_idx"][t].tolist()
        if policy == orc.SUBSTITUTION:
            want = r["assign"][t] + [-1] * (k - len(r["assign"][t]))
        else:
            keep = set(r["assign"][t])
            want = [i if i in keep else -1 for i in r["topk"][t]] + [-1] * (k - kk)
        assert got == want, f"assignment of token {t}: {got} vs {want}"
        for slot, i in enumerate(got):
            if i >= 0:
                assert g["tokslot2row"][t, slot] == r["row_of"][(t, i)], f"row of token {t} slot {slot}"
                w = r["wgt"][t, i]
                assert abs(g["gate_w"][t, slot] - w) <= 2e-7 * max(abs(w), 1e-30) + 1e-37, f"weight t={t} slot={slot}"
            else:
                assert g["tokslot2row"][t, slot] == -1 and g["gate_w"][t, slot] == 0.0
    assert g["count"] == r["count"] and g["offset"] == r["offset"]
    assert g["perm_row2tok"] == r["perm_row2tok"]
    # the GPU adds scores as 2^-52 fixed-point integers (order-independent): up to M half-ulps of 2^-52
    np.testing.assert_allclose(g["score"], r["score"], rtol=1e-12, atol=max(M, 1) * 2.0 ** -52)


def out_error(out_gpu, ref):
    """(max abs error, RMS of the reference)."""
    o = out_gpu.to("cpu", torch.float64).numpy()
    return float(np.max(np.abs(o - ref))) if ref.size else 0.0, float(np.sqrt(np.mean(ref ** 2))) if ref.size else 0.0

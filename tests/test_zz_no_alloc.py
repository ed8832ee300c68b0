"""moespec_route_static, the entry point for callers that cannot allocate device memory.

Such callers (code inside a CUDA stream capture, serving loops that must avoid the device-wide
synchronisation cudaMalloc can cause, processes whose memory belongs to another allocator) get the
routing step with its scratch in a fixed array inside the library.  This test calls it through the
C ABI twice in a row, with different sizes so that the second call sees the first call's leftovers
in the shared scratch, and requires the same results as the handle-based entry point.

The file sorts last on purpose: a run that stops at the first failure has then run everything else.
"""
import numpy as np
import pytest
import torch

from paper_2602_16052_b200 import synth

pytestmark = pytest.mark.gpu


def reference_routing(m, case, z, k, B, policy, shortlist, renorm):
    layer = m.Layer(case["router_w"], case["router_bias"], case["w_gate"], case["w_up"], case["w_down"],
                    max_M=z.shape[0], max_k=k, policy=policy, shortlist=shortlist, renormalize=renorm,
                    ffn_kernel=m.FFN_CUDA_CORE)
    layer.route_from_logits(z, k, B)
    g = layer.get_routing()
    layer.destroy()
    return g


def check_same(out, g, M, k):
    torch.cuda.synchronize()
    nS, _, R = out["summary"][:3].tolist()
    assert out["S_rank"][:nS].tolist() == g["S"] and R == g["n_rows"]
    for name in ("topk_idx", "assign_idx", "tokslot2row"):
        assert np.array_equal(out[name][:M * k].cpu().numpy().reshape(M, k), g[name]), name
    # same kernel, same inputs: the floating-point outputs are identical, which is inside any tolerance
    assert np.array_equal(out["gate_w"][:M * k].cpu().numpy().reshape(M, k), g["gate_w"])
    assert np.array_equal(out["score"].cpu().numpy(), g["score"])
    assert out["count"].tolist() == g["count"] and out["offset"].tolist() == g["offset"]
    assert out["perm_row2tok"][:R].tolist() == g["perm_row2tok"]


def test_route_static_matches_handle_based_routing_twice_in_a_row():
    from paper_2602_16052_b200 import moespec as m
    cfg = synth.CONFIGS["olmoe"].with_(f=128)
    case = synth.gen_layer(cfg, 21, 0, "cuda")
    k = cfg.k
    calls = [(127, 32, m.SUBSTITUTION, m.FROM_ALL, True), (40, 5, m.TRUNCATION, m.FROM_UNION, False),
             (300, 24, m.SUBSTITUTION, m.FROM_UNION, True), (9, 64, m.SUBSTITUTION, m.FROM_ALL, True)]
    for M, B, policy, shortlist, renorm in calls:
        h = synth.gen_hidden(cfg, M, 21, 0, "cuda")
        z = (h.float() @ case["router_w"].float().T + case["router_bias"]).contiguous()   # any fp32 logits will do
        want = reference_routing(m, case, z, k, B, policy, shortlist, renorm)
        got = m.route_static(z, k, B, policy, shortlist, renorm)
        check_same(got, want, M, k)
        again = m.route_static(z, k, B, policy, shortlist, renorm, out=got)     # reuse the caller's buffers
        check_same(again, want, M, k)


def test_route_static_large_tree_against_the_oracle():
    """Trees above 128 tokens take the branch in which a separate kernel works out the row of every (token,
    slot) pair from the bit matrix in the shared scratch.  Here the results are compared with the CPU oracle
    itself (a comparison with the handle-based entry point alone would pass a fault the two share), on a large
    call, then a small one that finds the large call's leftovers, then the large one again."""
    from oracle import moespec_oracle as orc
    from paper_2602_16052_b200 import moespec as m
    from tests import helpers as H
    cfg = synth.CONFIGS["olmoe"].with_(f=128)
    case = synth.gen_layer(cfg, 22, 0, "cpu")
    k = cfg.k
    calls = [(255, 32, orc.SUBSTITUTION, orc.FROM_ALL, True), (40, 12, orc.TRUNCATION, orc.FROM_UNION, False),
             (m.ROUTE_STATIC_MAX_M, 16, orc.TRUNCATION, orc.FROM_ALL, True), (255, 32, orc.SUBSTITUTION, orc.FROM_ALL, True)]
    for M, B, policy, shortlist, renorm in calls:
        h = synth.gen_hidden(cfg, M, 22, 0, "cpu")
        z = orc.router_logits(H.f64(h), H.f64(case["router_w"]), H.f64(case["router_bias"]))      # fp32 logits
        r = orc.route(z, k, B, policy, shortlist, renorm)
        got = m.route_static(torch.from_numpy(z).cuda(), k, B, policy, shortlist, renorm)
        torch.cuda.synchronize()
        nS, n_act, R = got["summary"][:3].tolist()
        g = {"S": got["S_rank"][:nS].tolist(), "n_rows": R, "count": got["count"].tolist(),
             "offset": got["offset"].tolist(), "perm_row2tok": got["perm_row2tok"][:R].tolist(),
             "score": got["score"].cpu().numpy()}
        for name in ("topk_idx", "assign_idx", "tokslot2row", "gate_w"):
            g[name] = got[name][:M * k].cpu().numpy().reshape(M, k)
        H.compare_routing(g, r, policy, k)
        assert n_act == len(r["active"]) and R == len(r["perm_row2tok"])


def test_route_static_replayed_from_a_captured_graph():
    """One of the callers this entry point is for runs inside a stream capture.  The first call on the device is
    made outside the capture (it looks up the scratch array's address); a later call is then captured into a
    CUDA graph and the graph is replayed on new logits: every replay must give the handle-based results."""
    from paper_2602_16052_b200 import moespec as m
    cfg = synth.CONFIGS["olmoe"].with_(f=128)
    case = synth.gen_layer(cfg, 23, 0, "cuda")
    k, M, B = cfg.k, 200, 20
    mk_logits = lambda seed: (synth.gen_hidden(cfg, M, seed, 0, "cuda").float() @ case["router_w"].float().T
                              + case["router_bias"]).contiguous()
    z = mk_logits(23)
    out = m.route_static(z, k, B, m.SUBSTITUTION, m.FROM_ALL, True)           # first call: outside any capture
    torch.cuda.synchronize()
    side = torch.cuda.Stream()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=side):
        m.route_static(z, k, B, m.SUBSTITUTION, m.FROM_ALL, True, out=out, stream=torch.cuda.current_stream())
    for seed in (24, 25):
        z.copy_(mk_logits(seed))
        torch.cuda.synchronize()
        g.replay()
        torch.cuda.synchronize()
        want = reference_routing(m, case, z, k, B, m.SUBSTITUTION, m.FROM_ALL, True)
        check_same(out, want, M, k)


def test_route_static_rejects_sizes_beyond_its_scratch():
    from paper_2602_16052_b200 import moespec as m
    z = torch.zeros((m.ROUTE_STATIC_MAX_M + 1, 8), dtype=torch.float32, device="cuda")
    with pytest.raises(m.MoeSpecError) as e:
        m.route_static(z, 2, 4, m.SUBSTITUTION, m.FROM_ALL, True)
    assert e.value.code == m.ERR_TOO_LARGE and "capacity" in str(e.value)
    z = torch.zeros((4, m.ROUTE_STATIC_MAX_N + 1), dtype=torch.float32, device="cuda")
    with pytest.raises(m.MoeSpecError) as e:
        m.route_static(z, 2, 4, m.SUBSTITUTION, m.FROM_ALL, True)
    assert e.value.code == m.ERR_TOO_LARGE

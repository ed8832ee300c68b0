"""Runs first among the GPU tests (the file name sorts first) and launches nothing but the library's own kernels:
the inputs of one small layer are generated on the CPU and uploaded, the layer runs through the C ABI and is
checked against the oracle.  A record of the first kernels this test process launches therefore shows the
layer's kernels, not an input generator's."""
import numpy as np
import pytest
import torch

from oracle import moespec_oracle as orc
from paper_2602_16052_b200 import synth

pytestmark = pytest.mark.gpu


def test_first_launches_are_the_layers_own_kernels():
    from paper_2602_16052_b200 import moespec as m
    cfg = synth.CONFIGS["olmoe"].with_(f=256, n_experts=32)
    M, B = 63, 12
    L = {name: t.cuda() for name, t in synth.gen_layer(cfg, 0, 0, "cpu").items()}
    h = synth.gen_hidden(cfg, M, 0, 0, "cpu").cuda()
    out = torch.empty((M, cfg.d), dtype=torch.float32, device="cuda")      # allocation only: no kernel
    layer = m.Layer(L["router_w"], L["router_bias"], L["w_gate"], L["w_up"], L["w_down"], max_M=M, max_k=cfg.k,
                    out_dtype=torch.float32)
    layer.verify_layer(h, cfg.k, B, out)       # router_topk_kernel, route_kernel, gather_rows_kernel, ffn_tc_kernel
    torch.cuda.synchronize()
    assert layer.last_launch_count() == 4 and layer.get_stats()["status"] == 0
    f64 = lambda t: t.to("cpu", torch.float64).numpy()
    ref = orc.verify_layer(f64(h), f64(L["router_w"]), f64(L["router_bias"]), f64(L["w_gate"]), f64(L["w_up"]),
                           f64(L["w_down"]), cfg.k, B, orc.SUBSTITUTION, orc.FROM_ALL, True, logits=layer.get_logits())
    g = layer.get_routing()
    assert g["S"] == ref["S"] and g["perm_row2tok"] == ref["perm_row2tok"]
    err = float(np.max(np.abs(f64(out) - ref["out"])))
    assert err <= 2e-2 * float(np.sqrt(np.mean(ref["out"] ** 2)))
    layer.destroy()

"""Seeded synthetic inputs for the budgeted MoE verify layer.

This module only makes inputs.  It holds none of the method's arithmetic (no
router, softmax, selection or FFN code) and is the one module that both the CPU
oracle's tests and the CUDA path's tests/bench import.  It imports neither.

Every tensor is a pure function of (seed, tensor id, layer, element index): a
counter-based generator built on the splitmix64 finaliser, written with integer
tensor ops that give the same bits on CPU and on CUDA, so any slice (one
expert's weights, one token's row) can be regenerated on either side without
materialising the rest.

Normal variates are Irwin-Hall sums: 12 independent 16-bit uniforms are added
as integers, centred and divided by 2**16.  The sum of 12 uniforms on
{0..65535} has standard deviation sqrt(65536**2 - 1) ~ 65536, so the value is a
unit-variance bell truncated at +-6 sigma, exactly representable in fp32.  One
fp32 multiply by sigma and one rounding to the storage dtype follow; both are
exactly rounded IEEE operations and therefore bit-identical on every device.

Shapes follow the three evaluated architectures (Section 4.1 "Models",
Table 3) and the tree sizes / budget ranges of Appendix A; the heavy-tailed
routing of Figure 2c is imitated with a router bias -slope * ln(rank_e), rank a
seeded permutation of 1..N.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace
from typing import Iterable, Optional, Sequence, Tuple

import torch

# tensor ids (part of the generator's key)
T_HIDDEN, T_ROUTER, T_RANK, T_W_GATE, T_W_UP, T_W_DOWN = 1, 2, 3, 4, 5, 6

_MASK64 = (1 << 64) - 1
_GAMMA = 0x9E3779B97F4A7C15
_MUL1 = 0xBF58476D1CE4E5B9
_MUL2 = 0x94D049BB133111EB
_IH_MEAN = 12 * 65535 // 2  # 393210, mean of the sum of 12 uniforms on {0..65535}


def _s64(x: int) -> int:
    """Two's-complement view of a 64-bit pattern as a signed Python int."""
    x &= _MASK64
    return x - (1 << 64) if x >> 63 else x


def splitmix64_int(x: int) -> int:
    """splitmix64 finaliser on a Python int (the scalar definition of the hash)."""
    z = (x + _GAMMA) & _MASK64
    z = ((z ^ (z >> 30)) * _MUL1) & _MASK64
    z = ((z ^ (z >> 27)) * _MUL2) & _MASK64
    return z ^ (z >> 31)


def stream_key(seed: int, tensor_id: int, layer: int) -> int:
    """64-bit key of one tensor's random stream."""
    k = splitmix64_int(seed & _MASK64)
    k = splitmix64_int(k ^ (tensor_id & _MASK64))
    k = splitmix64_int(k ^ (layer & _MASK64))
    return k


def _lsr(x: torch.Tensor, r: int) -> torch.Tensor:
    """Logical right shift of int64 bit patterns."""
    return (x >> r) & ((1 << (64 - r)) - 1)


def _splitmix64_t(x: torch.Tensor) -> torch.Tensor:
    """splitmix64 finaliser on int64 tensors (wrapping arithmetic)."""
    z = x + _s64(_GAMMA)
    z = (z ^ _lsr(z, 30)) * _s64(_MUL1)
    z = (z ^ _lsr(z, 27)) * _s64(_MUL2)
    return z ^ _lsr(z, 31)


def irwin_hall_int(key: int, start: int, count: int, device="cpu") -> torch.Tensor:
    """Centred integer Irwin-Hall sums n_e for elements e = start .. start+count-1.

    n_e = sum of the twelve 16-bit fields of hash(key + 3e + j), j = 0, 1, 2,
    minus 393210.  n_e / 65536 is the unit-variance normal variate.
    """
    e = torch.arange(start, start + count, dtype=torch.int64, device=device)
    base = e * 3 + _s64(key)
    total = torch.zeros(count, dtype=torch.int64, device=device)
    for j in range(3):
        h = _splitmix64_t(base + j)
        total += (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + ((h >> 48) & 0xFFFF)
    return total - _IH_MEAN


def irwin_hall_int_scalar(key: int, e: int) -> int:
    """Pure-Python definition of one element of `irwin_hall_int` (used to pin it)."""
    total = 0
    for j in range(3):
        h = splitmix64_int((key + 3 * e + j) & _MASK64)
        total += (h & 0xFFFF) + ((h >> 16) & 0xFFFF) + ((h >> 32) & 0xFFFF) + ((h >> 48) & 0xFFFF)
    return total - _IH_MEAN


_CHUNK = 1 << 24


def normal_fp32(key: int, start: int, count: int, sigma: float, device="cpu") -> torch.Tensor:
    """fp32 values sigma_fp32 * (n_e / 65536): one exactly rounded multiply per element."""
    out = torch.empty(count, dtype=torch.float32, device=device)
    s32 = float(torch.tensor(sigma, dtype=torch.float32))
    for c0 in range(0, count, _CHUNK):
        c = min(_CHUNK, count - c0)
        n = irwin_hall_int(key, start + c0, c, device)
        out[c0:c0 + c] = (n.to(torch.float32) * (1.0 / 65536.0)) * s32
    return out


def torch_dtype(name: str) -> torch.dtype:
    return {"bf16": torch.bfloat16, "fp32": torch.float32, "fp16": torch.float16}[name]


@dataclass(frozen=True)
class LayerConfig:
    """Shape of one MoE layer plus the routing-tail slope of its synthetic router bias."""
    name: str
    d: int
    n_experts: int
    k: int
    f: int
    dtype: str          # storage dtype of weights, hidden and out: "bf16" | "fp16" | "fp32"
    slope: float        # router bias = -slope * ln(rank)
    n_layers: int = 1

    def with_(self, **kw) -> "LayerConfig":
        return replace(self, **kw)

    def expert_weight_bytes(self) -> int:
        w = 4 if self.dtype == "fp32" else 2
        return 3 * self.d * self.f * w


# The five workload shapes (tree sizes M and budgets B are per-run arguments).
CONFIGS = {
    "tiny":     LayerConfig("tiny", d=256, n_experts=16, k=4, f=128, dtype="fp32", slope=1.0),
    "olmoe":    LayerConfig("olmoe", d=2048, n_experts=64, k=8, f=1024, dtype="bf16", slope=1.0),
    "olmoe16":  LayerConfig("olmoe16", d=2048, n_experts=64, k=8, f=1024, dtype="bf16", slope=1.0, n_layers=16),
    "qwen3":    LayerConfig("qwen3", d=2048, n_experts=128, k=8, f=768, dtype="bf16", slope=1.2, n_layers=48),
    "mixtral":  LayerConfig("mixtral", d=4096, n_experts=8, k=2, f=14336, dtype="bf16", slope=0.5),
}
SWEEPS = {
    "tiny":    {"M": [15], "B": [8]},
    "olmoe":   {"M": [63], "B": [16, 32, 48, 64]},
    "olmoe16": {"M": [1, 7, 31, 63, 127, 255, 511], "B": [32, 64]},
    "qwen3":   {"M": [63, 127], "B": [32, 64, 128]},
    "mixtral": {"M": [15, 63], "B": [4, 6, 8]},
}


def gen_hidden(cfg: LayerConfig, M: int, seed: int, layer: int = 0, device="cpu") -> torch.Tensor:
    """hidden[M, d]: unit-variance bell, every row divided by its RMS, rounded to cfg.dtype.

    The row sum of squares is taken over the integer variates (exact, order
    independent); sqrt and the divisions are exactly rounded fp64 operations.
    """
    key = stream_key(seed, T_HIDDEN, layer)
    n = irwin_hall_int(key, 0, M * cfg.d, device).view(M, cfg.d)
    sumsq = (n * n).sum(dim=1, keepdim=True)                    # exact in int64
    rms = torch.sqrt(sumsq.to(torch.float64) / float(cfg.d))    # in units of 1/65536
    rms = torch.where(rms == 0, torch.ones_like(rms), rms)
    h = n.to(torch.float64) / rms
    return h.to(torch.float32).to(torch_dtype(cfg.dtype))


def rank_permutation(n_experts: int, seed: int, layer: int = 0) -> list:
    """rank[e] in 1..N: position of expert e when experts are sorted by a per-expert hash."""
    key = stream_key(seed, T_RANK, layer)
    order = sorted(range(n_experts), key=lambda e: (splitmix64_int((key + e) & _MASK64), e))
    rank = [0] * n_experts
    for pos, e in enumerate(order):
        rank[e] = pos + 1
    return rank


def gen_router(cfg: LayerConfig, seed: int, layer: int = 0, device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Router matrix Wr[N, d] ~ N(0, 1/d) in cfg.dtype and bias[N] = -slope * ln(rank) in fp32."""
    key = stream_key(seed, T_ROUTER, layer)
    w = normal_fp32(key, 0, cfg.n_experts * cfg.d, 1.0 / math.sqrt(cfg.d), device)
    w = w.view(cfg.n_experts, cfg.d).to(torch_dtype(cfg.dtype))
    rank = rank_permutation(cfg.n_experts, seed, layer)
    bias = torch.tensor([-cfg.slope * math.log(r) for r in rank], dtype=torch.float64)
    return w, bias.to(torch.float32).to(device)


def gen_expert_weights(cfg: LayerConfig, seed: int, layer: int = 0, device="cpu",
                       experts: Optional[Sequence[int]] = None, out=None):
    """(w_gate[E, f, d], w_up[E, f, d], w_down[E, d, f]) ~ N(0, 1/d) in cfg.dtype.

    `experts` selects a subset (rows of the result follow its order); None means
    all N.  `out`, if given, is a triple of preallocated tensors to fill.
    """
    ids = list(range(cfg.n_experts)) if experts is None else list(experts)
    per = cfg.f * cfg.d
    sigma = 1.0 / math.sqrt(cfg.d)
    dt = torch_dtype(cfg.dtype)
    shapes = ((cfg.f, cfg.d), (cfg.f, cfg.d), (cfg.d, cfg.f))
    if out is None:
        out = tuple(torch.empty((len(ids),) + s, dtype=dt, device=device) for s in shapes)
    for tid, dst, shp in zip((T_W_GATE, T_W_UP, T_W_DOWN), out, shapes):
        key = stream_key(seed, tid, layer)
        for row, e in enumerate(ids):
            dst[row].copy_(normal_fp32(key, e * per, per, sigma, device).view(shp))
    return out


def gen_layer(cfg: LayerConfig, seed: int, layer: int = 0, device="cpu", experts=None):
    """Dict with router_w, router_bias, w_gate, w_up, w_down for one layer."""
    rw, rb = gen_router(cfg, seed, layer, device)
    wg, wu, wd = gen_expert_weights(cfg, seed, layer, device, experts)
    return {"router_w": rw, "router_bias": rb, "w_gate": wg, "w_up": wu, "w_down": wd}

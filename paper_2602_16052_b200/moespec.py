"""Thin ctypes binding over libmoespec.so (argument marshalling only).

Names mirror the C ABI in include/moespec.h.  Every step of the layer runs in
the library's CUDA kernels; nothing here computes.  Importing this module
loads the library and raises if it has not been built: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("MOESPEC_LIB") or os.path.join(_HERE, "libmoespec.so")   # override for debug builds

BF16, FP32, FP16 = 1, 2, 3
_DTYPES = {torch.bfloat16: 1, torch.float32: 2, torch.float16: 3}
SUBSTITUTION, TRUNCATION = 1, 2
FROM_ALL, FROM_UNION, STATIC = 1, 2, 3
FFN_AUTO, FFN_CUDA_CORE, FFN_TENSOR_CORE = 0, 1, 2

OK = 0
ERR_INVALID_ARG, ERR_NULL_POINTER, ERR_UNSUPPORTED, ERR_OUT_OF_MEMORY = -1, -2, -3, -4
ERR_CUDA, ERR_TIMEOUT, ERR_INTERNAL, ERR_BAD_HANDLE, ERR_TOO_LARGE = -5, -6, -7, -8, -9
ROUTE_STATIC_MAX_M, ROUTE_STATIC_MAX_N, ROUTE_STATIC_MAX_K, ROUTE_STATIC_MAX_ROWS = 512, 256, 32, 8192

EXPORTS = [
    "moespec_layer_create", "moespec_verify_layer", "moespec_verify_layer_host",
    "moespec_calibrate", "moespec_get_static_counts", "moespec_set_static_ranking", "moespec_reset_calibration",
    "moespec_route_from_logits", "moespec_route_static", "moespec_get_routing", "moespec_get_logits", "moespec_get_intermediate", "moespec_get_stats",
    "moespec_debug_set_wait", "moespec_set_profiling", "moespec_get_kernel_times", "moespec_last_launch_count", "moespec_destroy",
    "moespec_stack_create", "moespec_verify_stack", "moespec_verify_stack_host", "moespec_stack_get_stream",
    "moespec_stack_set_graph", "moespec_stack_last_launch_count", "moespec_stack_destroy",
    "moespec_oracle_ranking", "moespec_get_gram", "moespec_reconstruction_error", "moespec_strerror", "moespec_last_cuda_error",
    "moespec_version",
]


class LayerDesc(C.Structure):
    _fields_ = [
        ("d", C.c_int), ("n_experts", C.c_int), ("f", C.c_int), ("max_M", C.c_int), ("max_k", C.c_int),
        ("dtype", C.c_int), ("out_dtype", C.c_int), ("policy", C.c_int), ("shortlist", C.c_int), ("renormalize", C.c_int),
        ("residual", C.c_int), ("ffn_kernel", C.c_int), ("device", C.c_int),
        ("router_w", C.c_void_p), ("router_bias", C.c_void_p),
        ("w_gate", C.c_void_p), ("w_up", C.c_void_p), ("w_down", C.c_void_p),
        ("resident_first", C.c_int), ("resident_count", C.c_int),
    ]


class Stats(C.Structure):
    _fields_ = [
        ("n_union", C.c_int), ("n_shortlist", C.c_int), ("n_active", C.c_int), ("n_rows", C.c_int),
        ("n_dropped", C.c_int), ("status", C.c_int), ("coverage", C.c_double), ("weight_bytes", C.c_longlong),
    ]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class MoeSpecError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().moespec_strerror(code).decode()
        cuda = lib().moespec_last_cuda_error() if code == ERR_CUDA else 0
        super().__init__(f"{where}: {msg} ({code})" + (f", cudaError {cuda}" if cuda else ""))


_lib = None


def lib() -> C.CDLL:
    """Load the library once.  Raises if it is missing: the layer has no other implementation."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is not built; run python -m paper_2602_16052_b200.build")
        L = C.CDLL(LIB_PATH)
        vp, ci = C.c_void_p, C.c_int
        L.moespec_layer_create.argtypes = [C.POINTER(LayerDesc), C.POINTER(vp)]
        L.moespec_verify_layer.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        L.moespec_verify_layer_host.argtypes = [vp, vp, ci, ci, ci, vp, vp]
        L.moespec_calibrate.argtypes = [vp, vp, ci, ci, vp]
        L.moespec_get_static_counts.argtypes = [vp, vp]
        L.moespec_set_static_ranking.argtypes = [vp, vp, ci]
        L.moespec_reset_calibration.argtypes = [vp]
        L.moespec_route_from_logits.argtypes = [vp, vp, ci, ci, ci, vp]
        L.moespec_route_static.argtypes = [vp] + [ci] * 7 + [vp] * 11
        L.moespec_get_routing.argtypes = [vp] + [vp] * 11
        L.moespec_get_logits.argtypes = [vp, vp]
        L.moespec_get_intermediate.argtypes = [vp, ci, vp, C.c_longlong]
        L.moespec_get_stats.argtypes = [vp, C.POINTER(Stats)]
        L.moespec_debug_set_wait.argtypes = [vp, C.c_longlong, ci]
        L.moespec_set_profiling.argtypes = [vp, ci]
        L.moespec_get_kernel_times.argtypes = [vp, vp, ci, vp]
        L.moespec_last_launch_count.argtypes = [vp]
        L.moespec_destroy.argtypes = [vp]
        L.moespec_stack_create.argtypes = [vp, ci, C.POINTER(vp)]
        L.moespec_verify_stack.argtypes = [vp, vp, ci, ci, vp, vp, vp]
        L.moespec_verify_stack_host.argtypes = [vp, vp, ci, ci, vp, vp, vp]
        L.moespec_stack_get_stream.argtypes = [vp, ci, vp]
        L.moespec_stack_set_graph.argtypes = [vp, ci]
        L.moespec_stack_last_launch_count.argtypes = [vp]
        L.moespec_stack_destroy.argtypes = [vp]
        L.moespec_oracle_ranking.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp, vp]
        L.moespec_get_gram.argtypes = [vp, vp]
        L.moespec_reconstruction_error.argtypes = [vp, vp, vp, ci, vp, vp, vp]
        L.moespec_strerror.argtypes = [ci]
        L.moespec_strerror.restype = C.c_char_p
        for name in EXPORTS:
            if getattr(L, name).restype is not C.c_char_p:
                getattr(L, name).restype = ci
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != OK:
        raise MoeSpecError(code, where)


def _np_ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _stream_ptr(stream) -> int:
    s = torch.cuda.current_stream() if stream is None else stream
    return s.cuda_stream


def route_static(logits: torch.Tensor, k: int, B: int, policy: int, shortlist: int, renormalize: bool,
                 out: Optional[dict] = None, stream=None) -> dict:
    """moespec_route_static: the routing step with no allocation inside the library.

    For callers that cannot allocate device memory at the call site (inside a
    stream capture, in a loop that must not trigger cudaMalloc's device-wide
    synchronisation, or when another allocator owns the device memory).  The
    output tensors are the caller's: pass the dict a previous call returned to
    reuse them, otherwise this wrapper makes them with torch before calling in.
    All calls share one fixed scratch array inside the library, so calls that
    overlap on the GPU race; M, N, k are capped (ROUTE_STATIC_MAX_*).
    """
    M, N = logits.shape
    assert logits.dtype == torch.float32 and logits.is_cuda and logits.is_contiguous()
    if out is None:
        dev = logits.device
        i32 = lambda n: torch.empty(max(n, 1), dtype=torch.int32, device=dev)
        out = {"S_rank": i32(N), "topk_idx": i32(M * k), "assign_idx": i32(M * k),
               "gate_w": torch.empty(max(M * k, 1), dtype=torch.float32, device=dev), "count": i32(N),
               "offset": i32(N + 1), "perm_row2tok": i32(M * k), "tokslot2row": i32(M * k),
               "score": torch.empty(N, dtype=torch.float64, device=dev), "summary": i32(8)}
    p = lambda name: out[name].data_ptr()
    _check(lib().moespec_route_static(logits.data_ptr(), M, N, k, B, policy, shortlist, int(renormalize),
                                      p("S_rank"), p("topk_idx"), p("assign_idx"), p("gate_w"), p("count"),
                                      p("offset"), p("perm_row2tok"), p("tokslot2row"), p("score"), p("summary"),
                                      _stream_ptr(stream)), "moespec_route_static")
    return out


class Layer:
    """One MoE layer handle: moespec_layer_create / moespec_verify_layer / moespec_destroy.

    Weight tensors are borrowed; this object keeps references so they outlive the handle.
    """

    def __init__(self, router_w, router_bias, w_gate, w_up, w_down, *, max_M: int, max_k: int,
                 policy: int = SUBSTITUTION, shortlist: int = FROM_ALL, renormalize: bool = True,
                 residual: bool = False, ffn_kernel: int = FFN_AUTO, out_dtype: Optional[torch.dtype] = None,
                 resident: Optional[tuple] = None):
        """resident = (first, count): this layer is an expert-parallel shard that holds the experts
        first .. first+count-1 only; w_gate / w_up / w_down are then THOSE experts' weights ([count, ...]) and
        verify_layer returns the shard's partial sum.  None: all N experts are here."""
        for t in (router_w, w_gate, w_up, w_down):
            if not (t.is_cuda and t.is_contiguous()):
                raise ValueError("weights must be contiguous CUDA tensors")
        N, d = router_w.shape
        f = w_gate.shape[1]
        E = N if resident is None else int(resident[1])
        if tuple(w_gate.shape) != (E, f, d) or tuple(w_up.shape) != (E, f, d) or tuple(w_down.shape) != (E, d, f):
            raise ValueError("weight shapes must be [E,f,d], [E,f,d], [E,d,f] with E the experts held here")
        dt = _DTYPES[router_w.dtype]
        if router_bias is not None:
            router_bias = router_bias.to(device=router_w.device, dtype=torch.float32).contiguous()
        self._keep = (router_w, router_bias, w_gate, w_up, w_down)
        self.d, self.N, self.f, self.max_M, self.max_k = d, N, f, max_M, max_k
        self.dtype = router_w.dtype
        self.out_dtype = out_dtype or router_w.dtype
        self.device = router_w.device
        desc = LayerDesc(d=d, n_experts=N, f=f, max_M=max_M, max_k=max_k, dtype=dt,
                         out_dtype=_DTYPES[self.out_dtype], policy=policy,
                         shortlist=shortlist, renormalize=int(renormalize), residual=int(residual),
                         ffn_kernel=ffn_kernel, device=router_w.device.index or 0,
                         router_w=router_w.data_ptr(),
                         router_bias=None if router_bias is None else router_bias.data_ptr(),
                         w_gate=w_gate.data_ptr(), w_up=w_up.data_ptr(), w_down=w_down.data_ptr(),
                         resident_first=0 if resident is None else int(resident[0]),
                         resident_count=0 if resident is None else int(resident[1]))
        h = C.c_void_p()
        _check(lib().moespec_layer_create(C.byref(desc), C.byref(h)), "moespec_layer_create")
        self._h = h
        self._last = (0, 0)

    # -- the hot path
    def verify_layer(self, hidden: torch.Tensor, k: int, B: int, out: Optional[torch.Tensor] = None, stream=None):
        M = hidden.shape[0]
        if out is None:
            out = torch.empty(hidden.shape, dtype=self.out_dtype, device=hidden.device)
        _check(lib().moespec_verify_layer(self._h, hidden.data_ptr(), M, k, B, out.data_ptr(), _stream_ptr(stream)),
               "moespec_verify_layer")
        self._last = (M, k)
        return out

    def verify_layer_host(self, hidden_host: torch.Tensor, k: int, B: int, out_host: torch.Tensor, stream=None):
        M = hidden_host.shape[0]
        _check(lib().moespec_verify_layer_host(self._h, hidden_host.data_ptr(), M, k, B, out_host.data_ptr(),
                                               _stream_ptr(stream)), "moespec_verify_layer_host")
        self._last = (M, k)
        return out_host

    # -- static ranking (Eq. 4)
    def calibrate(self, hidden: torch.Tensor, k: int, stream=None):
        M = hidden.shape[0]
        _check(lib().moespec_calibrate(self._h, hidden.data_ptr(), M, k, _stream_ptr(stream)), "moespec_calibrate")
        self._last = (M, k)

    def get_static_counts(self) -> np.ndarray:
        c = np.zeros(self.N, dtype=np.int64)
        _check(lib().moespec_get_static_counts(self._h, _np_ptr(c)), "moespec_get_static_counts")
        return c

    def set_static_ranking(self, ranked=None):
        if ranked is None:
            _check(lib().moespec_set_static_ranking(self._h, None, 0), "moespec_set_static_ranking")
        else:
            a = np.ascontiguousarray(ranked, dtype=np.int32)
            _check(lib().moespec_set_static_ranking(self._h, _np_ptr(a), len(a)), "moespec_set_static_ranking")

    def reset_calibration(self):
        _check(lib().moespec_reset_calibration(self._h), "moespec_reset_calibration")

    def route_from_logits(self, logits: torch.Tensor, k: int, B: int, stream=None):
        M = logits.shape[0]
        assert logits.dtype == torch.float32 and logits.is_cuda and logits.is_contiguous()
        _check(lib().moespec_route_from_logits(self._h, logits.data_ptr(), M, k, B, _stream_ptr(stream)),
               "moespec_route_from_logits")
        self._last = (M, k)

    # -- introspection
    def get_routing(self) -> dict:
        M, k = self._last
        N = self.N
        i32 = lambda n: np.full(max(n, 1), -7, dtype=np.int32)
        S, nS, nR = i32(N), C.c_int(0), C.c_int(0)
        topk, assign, slot2row = i32(M * k), i32(M * k), i32(M * k)
        gate = np.zeros(max(M * k, 1), dtype=np.float32)
        count, offset = i32(N), i32(N + 1)
        perm = i32(M * k)
        score = np.zeros(N, dtype=np.float64)
        _check(lib().moespec_get_routing(self._h, _np_ptr(S), C.cast(C.byref(nS), C.c_void_p), _np_ptr(topk),
                                         _np_ptr(assign), _np_ptr(gate), _np_ptr(count), _np_ptr(offset),
                                         _np_ptr(perm), _np_ptr(slot2row), _np_ptr(score),
                                         C.cast(C.byref(nR), C.c_void_p)), "moespec_get_routing")
        R = nR.value
        return {"S": S[:nS.value].tolist(), "topk_idx": topk[:M * k].reshape(M, k),
                "assign_idx": assign[:M * k].reshape(M, k), "gate_w": gate[:M * k].reshape(M, k),
                "count": count.tolist(), "offset": offset.tolist(), "perm_row2tok": perm[:R].tolist(),
                "tokslot2row": slot2row[:M * k].reshape(M, k), "score": score, "n_rows": R}

    def get_logits(self) -> np.ndarray:
        M, _ = self._last
        z = np.zeros((M, self.N), dtype=np.float32)
        _check(lib().moespec_get_logits(self._h, _np_ptr(z)), "moespec_get_logits")
        return z

    def get_intermediate(self, which: str, n_rows: int) -> torch.Tensor:
        """Host copy of x_perm [R,d], h_mid [R,f] (layer dtype) or y [R,d] (fp32) of the last call."""
        idx = {"x_perm": 0, "h_mid": 1, "y": 2}[which]
        cols = self.f if idx == 1 else self.d
        t = torch.empty((n_rows, cols), dtype=torch.float32 if idx == 2 else self.dtype)
        if n_rows:
            _check(lib().moespec_get_intermediate(self._h, idx, t.data_ptr(), t.numel() * t.element_size()),
                   "moespec_get_intermediate")
        return t

    def get_stats(self) -> dict:
        st = Stats()
        _check(lib().moespec_get_stats(self._h, C.byref(st)), "moespec_get_stats")
        return st.as_dict()

    KERNEL_NAMES_TC = ("router_topk", "route", "gather", "ffn")
    KERNEL_NAMES_TC_SMALL = ("router_topk", "route", "ffn")      # trees of at most 16 tokens: no gathered copy
    KERNEL_NAMES_CC = ("router_topk", "route", "gather", "ffn_gate_up", "ffn_down", "combine")

    def debug_set_wait(self, limit_cycles: int, ready_bias: int):
        """Test hook: bound of the device-side waits and a ready-counter bias that makes them run out."""
        _check(lib().moespec_debug_set_wait(self._h, limit_cycles, ready_bias), "moespec_debug_set_wait")

    def set_profiling(self, on: bool):
        _check(lib().moespec_set_profiling(self._h, int(on)), "moespec_set_profiling")

    def get_kernel_times(self) -> dict:
        """Milliseconds per kernel of the last verify call (profiling must be on)."""
        ms = (C.c_float * 8)()
        n = C.c_int(0)
        _check(lib().moespec_get_kernel_times(self._h, C.cast(ms, C.c_void_p), 8, C.cast(C.byref(n), C.c_void_p)),
               "moespec_get_kernel_times")
        names = {3: self.KERNEL_NAMES_TC_SMALL, 4: self.KERNEL_NAMES_TC}.get(n.value, self.KERNEL_NAMES_CC)
        return {names[i]: float(ms[i]) for i in range(min(n.value, len(names)))}

    def last_launch_count(self) -> int:
        return lib().moespec_last_launch_count(self._h)

    # -- analysis mode (Eq. 6, Section 4.5)
    def oracle_ranking(self, hidden: torch.Tensor, k: int, n_pick: int, out_star: Optional[torch.Tensor] = None,
                       stream=None):
        """Greedy oracle ordering: returns (order[n_pick], objective[n_pick], gold_energy)."""
        M = hidden.shape[0]
        order = np.zeros(n_pick, dtype=np.int32)
        obj = np.zeros(n_pick, dtype=np.float64)
        gold = np.zeros(1, dtype=np.float64)
        _check(lib().moespec_oracle_ranking(self._h, hidden.data_ptr(), M, k, n_pick, _np_ptr(order), _np_ptr(obj),
                                            _np_ptr(gold), None if out_star is None else out_star.data_ptr(),
                                            _stream_ptr(stream)), "moespec_oracle_ranking")
        self._last = (M, k)
        return order.tolist(), obj, float(gold[0])

    def get_gram(self) -> np.ndarray:
        M, k = self._last
        g = np.zeros((M, k, k), dtype=np.float64)
        _check(lib().moespec_get_gram(self._h, _np_ptr(g)), "moespec_get_gram")
        return g

    def reconstruction_error(self, out_S: torch.Tensor, out_star: torch.Tensor, stream=None):
        """(||O_S - O*||^2 / ||O*||^2, numerator, denominator)."""
        err = np.zeros(1, dtype=np.float64)
        sums = np.zeros(2, dtype=np.float64)
        _check(lib().moespec_reconstruction_error(self._h, out_S.data_ptr(), out_star.data_ptr(), out_S.shape[0],
                                                  _np_ptr(err), _np_ptr(sums), _stream_ptr(stream)),
               "moespec_reconstruction_error")
        return float(err[0]), float(sums[0]), float(sums[1])

    def destroy(self):
        if getattr(self, "_h", None) is not None and self._h:
            code = lib().moespec_destroy(self._h)
            self._h = None
            _check(code, "moespec_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass


class Stack:
    """L layers on one residual stream: moespec_stack_create / moespec_verify_stack / moespec_stack_destroy.

    The layers are borrowed (kept referenced here); each must have residual=True and out_dtype == dtype.
    """

    def __init__(self, layers):
        self.layers = list(layers)
        arr = (C.c_void_p * len(self.layers))(*[L._h for L in self.layers])
        h = C.c_void_p()
        _check(lib().moespec_stack_create(C.cast(arr, C.c_void_p), len(self.layers), C.byref(h)), "moespec_stack_create")
        self._h = h
        self._last_M = 0

    def _budgets(self, budgets):
        if isinstance(budgets, int):
            budgets = [budgets] * len(self.layers)
        if len(budgets) != len(self.layers):
            raise ValueError("one budget per layer")
        return (C.c_int * len(self.layers))(*[int(b) for b in budgets])

    def verify_stack(self, hidden: torch.Tensor, k: int, budgets, out: Optional[torch.Tensor] = None, stream=None):
        M = hidden.shape[0]
        if out is None:
            out = torch.empty_like(hidden)
        b = self._budgets(budgets)
        _check(lib().moespec_verify_stack(self._h, hidden.data_ptr(), M, k, C.cast(b, C.c_void_p), out.data_ptr(),
                                          _stream_ptr(stream)), "moespec_verify_stack")
        self._last_M = M
        for L in self.layers:
            L._last = (M, k)
        return out

    def verify_stack_host(self, hidden_host: torch.Tensor, k: int, budgets, out_host: torch.Tensor, stream=None):
        M = hidden_host.shape[0]
        b = self._budgets(budgets)
        _check(lib().moespec_verify_stack_host(self._h, hidden_host.data_ptr(), M, k, C.cast(b, C.c_void_p),
                                               out_host.data_ptr(), _stream_ptr(stream)), "moespec_verify_stack_host")
        self._last_M = M
        for L in self.layers:
            L._last = (M, k)
        return out_host

    def get_stream(self, l: int) -> torch.Tensor:
        """x_l of the last pass (1 <= l <= L-1) as a CPU tensor [M, d]."""
        x = torch.empty((self._last_M, self.layers[0].d), dtype=self.layers[0].dtype)
        _check(lib().moespec_stack_get_stream(self._h, l, x.data_ptr()), "moespec_stack_get_stream")
        return x

    def set_graph(self, on: bool):
        _check(lib().moespec_stack_set_graph(self._h, int(on)), "moespec_stack_set_graph")

    def last_launch_count(self) -> int:
        return lib().moespec_stack_last_launch_count(self._h)

    def destroy(self):
        if getattr(self, "_h", None) is not None and self._h:
            code = lib().moespec_stack_destroy(self._h)
            self._h = None
            _check(code, "moespec_stack_destroy")

    def __del__(self):
        try:
            self.destroy()
        except Exception:
            pass

"""Thin ctypes binding over libd2d.so (the C ABI of include/d2d.h).

Argument marshalling only: every step of the layer runs inside the CUDA library.
PyTorch is used for device memory and streams.  Importing this module loads the
library and raises if it has not been built (`python -m paper_2310_04361_b200.build`);
there is no CPU fallback.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import POINTER, c_char_p, c_float, c_int, c_int32, c_int64, c_size_t, c_void_p

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libd2d.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2310_04361_b200.build` "
                      "(the dynamic-k MoE layer has no CPU fallback)")
_lib = ctypes.CDLL(LIB_PATH)

D2D_OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "WORKSPACE", 4: "CUDA", 5: "NONFINITE",
                6: "TIMEOUT", 7: "CAPACITY"}
D2D_F32, D2D_BF16 = 0, 1
ACTS = {"relu": 0, "gelu_erf": 1, "gelu_tanh": 2, "silu": 3}
PATHS = {"auto": 0, "dense": 1, "gather": 2, "fused": 3}
EXPORTS = ["d2d_status_str", "d2d_launch_count", "d2d_layer_create", "d2d_layer_create_fp8", "d2d_layer_get_fp8", "d2d_layer_destroy", "d2d_workspace_bytes",
           "d2d_layer_set_expert_path", "d2d_layer_set_fused_rho_max", "d2d_layer_get_fused", "d2d_layer_expert_path_for", "d2d_layer_get_expert_path", "d2d_layer_reset_counters", "d2d_expert_up_gather_fwd", "d2d_expert_down_masked_fwd", "d2d_test_inject_fault",
           "d2d_select_workspace_bytes", "d2d_router_fwd", "d2d_select_dynk", "d2d_select_dynk_static", "d2d_select_topk",
           "d2d_routing_from_mask", "d2d_moe_ffn_fwd", "d2d_expert_up_fwd", "d2d_expert_down_fwd", "d2d_layer_fwd", "d2d_layer_fwd_host_workspace_bytes",
           "d2d_layer_fwd_host", "d2d_group_create", "d2d_group_destroy", "d2d_group_workspace_bytes", "d2d_group_fwd"]


class LayerDesc(ctypes.Structure):
    _fields_ = [("d", c_int32), ("d_ff", c_int32), ("n_experts", c_int32), ("expert_size", c_int32),
                ("d_h", c_int32), ("dtype", c_int), ("act", c_int), ("gated", c_int32)]


class Weights(ctypes.Structure):
    _fields_ = [(n, c_void_p) for n in ("w_r1", "b_r1", "w_r2", "b_r2", "w1", "b1", "w_gate", "w2", "b2")]


class RoutingStruct(ctypes.Structure):
    _fields_ = [("mask", c_void_p), ("k", c_void_p), ("counts", c_void_p), ("offsets", c_void_p),
                ("perm", c_void_p), ("tok_off", c_void_p), ("tok_exp", c_void_p), ("n_sel", c_void_p),
                ("status", c_void_p), ("perm_capacity", c_int64)]


_lib.d2d_launch_count.restype = ctypes.c_uint64
_lib.d2d_launch_count.argtypes = []
_lib.d2d_status_str.restype = c_char_p
_lib.d2d_status_str.argtypes = [c_int]
_lib.d2d_layer_create.argtypes = [POINTER(LayerDesc), POINTER(Weights), c_void_p, POINTER(c_void_p)]
_lib.d2d_layer_create_fp8.argtypes = [POINTER(LayerDesc), POINTER(Weights), c_void_p, POINTER(c_void_p)]
_lib.d2d_layer_get_fp8.argtypes = [c_void_p, c_int32, c_void_p, c_void_p, c_void_p]
_lib.d2d_layer_destroy.argtypes = [c_void_p]
_lib.d2d_workspace_bytes.restype = c_size_t
_lib.d2d_workspace_bytes.argtypes = [c_void_p, c_int32]
_lib.d2d_select_workspace_bytes.restype = c_size_t
_lib.d2d_select_workspace_bytes.argtypes = [c_int32, c_int32]
_lib.d2d_router_fwd.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_size_t, c_void_p]
_lib.d2d_select_dynk.argtypes = [c_void_p, c_int32, c_int32, c_float, POINTER(RoutingStruct), c_void_p, c_size_t, c_void_p]
_lib.d2d_select_dynk_static.argtypes = [c_void_p, c_int32, c_int32, c_float, POINTER(RoutingStruct), c_void_p]
_lib.d2d_select_topk.argtypes = [c_void_p, c_int32, c_int32, c_int32, POINTER(RoutingStruct), c_void_p, c_size_t, c_void_p]
_lib.d2d_routing_from_mask.argtypes = [c_int32, c_int32, POINTER(RoutingStruct), c_void_p, c_size_t, c_void_p]
_lib.d2d_moe_ffn_fwd.argtypes = [c_void_p, c_void_p, c_int32, POINTER(RoutingStruct), c_void_p, c_void_p, c_size_t, c_void_p]
_lib.d2d_expert_up_fwd.argtypes = [c_void_p, c_void_p, c_int32, POINTER(RoutingStruct), c_void_p, c_void_p]
_lib.d2d_expert_up_gather_fwd.argtypes = [c_void_p, c_void_p, c_int32, POINTER(RoutingStruct), c_void_p, c_void_p]
_lib.d2d_expert_down_masked_fwd.argtypes = [c_void_p, c_void_p, c_int32, POINTER(RoutingStruct), c_void_p, c_void_p]
_lib.d2d_layer_set_expert_path.argtypes = [c_void_p, c_int, c_int32, ctypes.c_double]
_lib.d2d_layer_set_fused_rho_max.argtypes = [c_void_p, ctypes.c_double]
_lib.d2d_layer_get_fused.argtypes = [c_void_p, POINTER(c_int32), POINTER(ctypes.c_double)]
_lib.d2d_layer_expert_path_for.argtypes = [c_void_p, c_int32, ctypes.c_int64, POINTER(c_int32)]
_lib.d2d_layer_get_expert_path.argtypes = [c_void_p, POINTER(c_int32), POINTER(c_int32), POINTER(ctypes.c_double)]
_lib.d2d_layer_reset_counters.argtypes = [c_void_p, c_void_p]
_lib.d2d_test_inject_fault.argtypes = [c_int32]
_lib.d2d_expert_down_fwd.argtypes = [c_void_p, c_void_p, c_int32, c_void_p, c_void_p, c_void_p]
_lib.d2d_layer_fwd.argtypes = [c_void_p, c_void_p, c_int32, c_float, c_void_p, c_void_p, POINTER(RoutingStruct),
                               c_void_p, c_size_t, c_void_p]
_lib.d2d_layer_fwd_host_workspace_bytes.restype = c_size_t
_lib.d2d_layer_fwd_host_workspace_bytes.argtypes = [c_void_p, c_int32]
_lib.d2d_layer_fwd_host.argtypes = [c_void_p, c_void_p, c_int32, c_float, c_void_p, c_void_p, c_size_t, c_void_p]
_lib.d2d_group_create.argtypes = [POINTER(c_void_p), c_int32, c_void_p, POINTER(c_void_p)]
_lib.d2d_group_destroy.argtypes = [c_void_p]
_lib.d2d_group_workspace_bytes.restype = c_size_t
_lib.d2d_group_workspace_bytes.argtypes = [c_void_p, c_int32]
_lib.d2d_group_fwd.argtypes = [c_void_p, c_void_p, c_int32, c_float, c_void_p, POINTER(RoutingStruct), c_void_p, c_size_t,
                               c_void_p]


def launch_count() -> int:
    """Kernels launched by the library in this process so far."""
    return int(_lib.d2d_launch_count())


class D2DError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS_NAMES.get(code, code)} ({_lib.d2d_status_str(code).decode()})")


def _check(code: int, where: str) -> None:
    if code != D2D_OK:
        raise D2DError(code, where)


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return c_void_p(s.cuda_stream)


def torch_dtype(name: str):
    return torch.float32 if name == "f32" else torch.bfloat16


class Routing:
    """Caller-owned device buffers for the routing of one batch (d2d_routing)."""

    def __init__(self, T: int, E: int, device, dual: bool = False, perm_capacity: int | None = None, lists: bool = True):
        """lists=False leaves out the per-expert lists (counts, offsets, perm, n_sel): d2d_layer_fwd then does not build them."""
        W = (E + 31) // 32
        cap = T * E if perm_capacity is None else int(perm_capacity)
        i32 = dict(dtype=torch.int32, device=device)
        self.T, self.E, self.W = T, E, W
        self.mask = torch.zeros((max(T, 1), W), **i32)     # raw uint32 words kept in an int32 tensor
        self.k = torch.zeros((max(T, 1),), **i32)
        self.scalars = torch.zeros((2,), **i32)            # n_sel, status
        self.lists = lists
        if not lists:
            self.counts = self.offsets = self.perm = self.tok_off = self.tok_exp = None
            self.struct = RoutingStruct(mask=self.mask.data_ptr(), k=self.k.data_ptr(), counts=None, offsets=None, perm=None,
                                        tok_off=None, tok_exp=None, n_sel=None, status=self.scalars.data_ptr() + 4,
                                        perm_capacity=0)
            return
        self.counts = torch.zeros((E,), **i32)
        self.offsets = torch.zeros((E + 1,), **i32)
        self.perm = torch.zeros((max(cap, 1),), **i32)
        self.tok_off = torch.zeros((T + 1,), **i32) if dual else None
        self.tok_exp = torch.zeros((max(cap, 1),), **i32) if dual else None
        self.struct = RoutingStruct(
            mask=self.mask.data_ptr(), k=self.k.data_ptr(), counts=self.counts.data_ptr(),
            offsets=self.offsets.data_ptr(), perm=self.perm.data_ptr(),
            tok_off=self.tok_off.data_ptr() if dual else None,
            tok_exp=self.tok_exp.data_ptr() if dual else None,
            n_sel=self.scalars.data_ptr(), status=self.scalars.data_ptr() + 4, perm_capacity=cap)

    @property
    def n_sel(self) -> int:
        """Selected (token, expert) pairs: the library's n_sel, or the sum of k when the lists were not built."""
        if not self.lists:
            return int(self.k[: self.T].sum().item())
        return int(self.scalars[0].item())

    @property
    def status(self) -> int:
        return int(self.scalars[1].item())

    def mask_u32(self):
        """Mask words as a numpy uint32 array [T, W]."""
        return self.mask[: self.T].cpu().numpy().view("uint32")


class Layer:
    """One D2DMoE layer: packed device weights plus the calls of the C ABI."""

    def __init__(self, d: int, d_ff: int, n_experts: int, d_h: int, dtype: str, act: str, gated: bool,
                 weights: dict, device="cuda:0", fp8_experts: bool = False):
        self.device = torch.device(device)
        self.dtype_name = dtype
        self.tdtype = torch_dtype(dtype)
        self.d, self.d_ff, self.E, self.d_h = d, d_ff, n_experts, d_h
        self.s = d_ff // n_experts
        self.desc = LayerDesc(d=d, d_ff=d_ff, n_experts=n_experts, expert_size=self.s, d_h=d_h,
                              dtype=D2D_F32 if dtype == "f32" else D2D_BF16, act=ACTS[act], gated=int(bool(gated)))
        dev = {}
        for name in ("w_r1", "b_r1", "w_r2", "b_r2", "w1", "b1", "w_gate", "w2", "b2"):
            v = weights.get(name)
            if v is not None:
                t = v if isinstance(v, torch.Tensor) else torch.from_numpy(v)
                dev[name] = t.to(device=self.device, dtype=self.tdtype).contiguous()
        w = Weights(**{n: (dev[n].data_ptr() if n in dev else None) for n, _ in Weights._fields_})
        handle = c_void_p()
        with torch.cuda.device(self.device):
            create = _lib.d2d_layer_create_fp8 if fp8_experts else _lib.d2d_layer_create
            _check(create(ctypes.byref(self.desc), ctypes.byref(w), _stream(), ctypes.byref(handle)),
                   "d2d_layer_create_fp8" if fp8_experts else "d2d_layer_create")
        self.handle = handle
        self.fp8_experts = bool(fp8_experts)
        self._ws = None

    @classmethod
    def from_config(cls, cfg, weights: dict, device="cuda:0", fp8_experts: bool = False) -> "Layer":
        return cls(cfg.d, cfg.d_ff, cfg.E, cfg.d_h, cfg.dtype, cfg.act, cfg.gated, weights, device, fp8_experts)

    def get_fp8(self, which: str):
        """Codes (uint8 [d_ff, d]; "w2": of the transposed W2) and scale exponents (int32 [E]) of "w1" | "w_gate" | "w2"."""
        codes = torch.empty((self.d_ff, self.d), dtype=torch.uint8, device=self.device)
        exps = torch.empty((self.E,), dtype=torch.int32, device=self.device)
        _check(_lib.d2d_layer_get_fp8(self.handle, {"w1": 0, "w_gate": 1, "w2": 2}[which], _ptr(codes), _ptr(exps), _stream()),
               "d2d_layer_get_fp8")
        return codes, exps

    def close(self):
        if getattr(self, "handle", None):
            _lib.d2d_layer_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- workspace -------------------------------------------------------------------------
    def workspace_bytes(self, T: int) -> int:
        return int(_lib.d2d_workspace_bytes(self.handle, T))

    def workspace(self, T: int):
        need = self.workspace_bytes(T)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty((need,), dtype=torch.uint8, device=self.device)
        return self._ws

    def new_routing(self, T: int, dual: bool = False, perm_capacity: int | None = None, lists: bool = True) -> Routing:
        return Routing(T, self.E, self.device, dual, perm_capacity, lists)

    # -- which up projection the tensor-core expert step uses --------------------------------
    def set_expert_path(self, path: str = "auto", group: int = 0, rho_max: float = -1.0) -> None:
        """path: "auto" | "dense" | "gather"; group: experts per group (0 = default); rho_max: crossover density of
        "auto" (negative = default).  See d2d_layer_set_expert_path."""
        _check(_lib.d2d_layer_set_expert_path(self.handle, PATHS[path], int(group), float(rho_max)), "d2d_layer_set_expert_path")

    def set_fused_rho_max(self, rho_max: float = -1.0) -> None:
        """Density up to which "auto" takes the fused gathered kernel (negative = default, 0 = never)."""
        _check(_lib.d2d_layer_set_fused_rho_max(self.handle, float(rho_max)), "d2d_layer_set_fused_rho_max")

    def expert_path_for(self, T: int, n_sel: int) -> str:
        """The form of the expert step a call with T tokens and n_sel selected pairs takes ("dense" | "gather" | "fused")."""
        path = c_int32()
        _check(_lib.d2d_layer_expert_path_for(self.handle, int(T), int(n_sel), ctypes.byref(path)), "d2d_layer_expert_path_for")
        return {v: k for k, v in PATHS.items()}[path.value]

    def get_fused(self):
        group, rho = c_int32(), ctypes.c_double()
        _check(_lib.d2d_layer_get_fused(self.handle, ctypes.byref(group), ctypes.byref(rho)), "d2d_layer_get_fused")
        return group.value, rho.value

    def get_expert_path(self):
        path, group, rho = c_int32(), c_int32(), ctypes.c_double()
        _check(_lib.d2d_layer_get_expert_path(self.handle, ctypes.byref(path), ctypes.byref(group), ctypes.byref(rho)),
               "d2d_layer_get_expert_path")
        return {v: k for k, v in PATHS.items()}[path.value], group.value, rho.value

    def reset_counters(self, stream=None) -> None:
        _check(_lib.d2d_layer_reset_counters(self.handle, _stream(stream)), "d2d_layer_reset_counters")

    # -- the calls of the C ABI -------------------------------------------------------------
    def router_fwd(self, x, R=None, stream=None):
        T = x.shape[0]
        if R is None:
            R = torch.empty((T, self.E), dtype=torch.float32, device=self.device)
        ws = self.workspace(T)
        _check(_lib.d2d_router_fwd(self.handle, _ptr(x), T, _ptr(R), _ptr(ws), ws.numel(), _stream(stream)),
               "d2d_router_fwd")
        return R

    def moe_ffn_fwd(self, x, routing: Routing, y=None, stream=None):
        T = x.shape[0]
        if y is None:
            y = torch.empty((T, self.d), dtype=self.tdtype, device=self.device)
        ws = self.workspace(T)
        _check(_lib.d2d_moe_ffn_fwd(self.handle, _ptr(x), T, ctypes.byref(routing.struct), _ptr(y), _ptr(ws),
                                    ws.numel(), _stream(stream)), "d2d_moe_ffn_fwd")
        return y

    def expert_up_fwd(self, x, routing: Routing, H=None, stream=None):
        """H = mask * A(x W1^T + b1), bf16 [T, d_ff] (the tensor-core up projection on its own)."""
        T = x.shape[0]
        if H is None:
            H = torch.empty((T, self.d_ff), dtype=torch.bfloat16, device=self.device)
        _check(_lib.d2d_expert_up_fwd(self.handle, _ptr(x), T, ctypes.byref(routing.struct), _ptr(H), _stream(stream)),
               "d2d_expert_up_fwd")
        return H

    def expert_down_masked_fwd(self, H, routing: Routing, y=None, stream=None):
        """y = (G * H) W2^T + b2, reading only the kept cells of H (the down projection after the gathered kernel)."""
        T = H.shape[0]
        if y is None:
            y = torch.empty((T, self.d), dtype=torch.bfloat16, device=self.device)
        _check(_lib.d2d_expert_down_masked_fwd(self.handle, _ptr(H), T, ctypes.byref(routing.struct), _ptr(y), _stream(stream)),
               "d2d_expert_down_masked_fwd")
        return y

    def expert_up_gather_fwd(self, x, routing: Routing, H=None, stream=None):
        """The gathered, grouped kernel (tokens bucketed by groups of adjacent experts): writes only the kept
        (token, group) cells of H, the same values expert_up_fwd writes there."""
        T = x.shape[0]
        if H is None:
            H = torch.empty((T, self.d_ff), dtype=torch.bfloat16, device=self.device)
        _check(_lib.d2d_expert_up_gather_fwd(self.handle, _ptr(x), T, ctypes.byref(routing.struct), _ptr(H), _stream(stream)),
               "d2d_expert_up_gather_fwd")
        return H

    def expert_down_fwd(self, H, y=None, stream=None):
        """y = H W2^T + b2, bf16 [T, d] (the tensor-core down projection on its own)."""
        T = H.shape[0]
        if y is None:
            y = torch.empty((T, self.d), dtype=torch.bfloat16, device=self.device)
        _check(_lib.d2d_expert_down_fwd(self.handle, _ptr(H), T, _ptr(y), None, _stream(stream)), "d2d_expert_down_fwd")
        return y

    def layer_fwd(self, x, tau: float, y=None, routing: Routing | None = None, R_out=None, stream=None):
        T = x.shape[0]
        if y is None:
            y = torch.empty((T, self.d), dtype=self.tdtype, device=self.device)
        if routing is None:
            routing = self.new_routing(T)
        ws = self.workspace(T)
        _check(_lib.d2d_layer_fwd(self.handle, _ptr(x), T, c_float(tau), _ptr(y), _ptr(R_out),
                                  ctypes.byref(routing.struct), _ptr(ws), ws.numel(), _stream(stream)),
               "d2d_layer_fwd")
        return y, routing

    def host_workspace(self, T: int):
        need = int(_lib.d2d_layer_fwd_host_workspace_bytes(self.handle, T))
        return torch.empty((need,), dtype=torch.uint8, device=self.device)

    def layer_fwd_host(self, x_host, tau: float, y_host, ws, stream=None):
        """x_host / y_host: CPU tensors [T,d] of the layer dtype (pinned for speed); synchronises the stream."""
        T = x_host.shape[0]
        _check(_lib.d2d_layer_fwd_host(self.handle, c_void_p(x_host.data_ptr()), T, c_float(tau),
                                       c_void_p(y_host.data_ptr()), _ptr(ws), ws.numel(), _stream(stream)),
               "d2d_layer_fwd_host")
        return y_host


class LayerGroup:
    """Layers of one shape that read the same tokens (the Q, K and V projections of an attention layer): d2d_group_*."""

    def __init__(self, layers: list):
        self.layers = list(layers)                      # the group does not own the layers: keep them alive
        self.device = self.layers[0].device if self.layers else torch.device("cuda:0")
        arr = (c_void_p * len(self.layers))(*[l.handle for l in self.layers])
        handle = c_void_p()
        with torch.cuda.device(self.device):
            _check(_lib.d2d_group_create(arr, len(self.layers), _stream(), ctypes.byref(handle)), "d2d_group_create")
        self.handle = handle
        self._ws = None

    def close(self):
        if getattr(self, "handle", None):
            _lib.d2d_group_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def workspace(self, T: int):
        need = int(_lib.d2d_group_workspace_bytes(self.handle, T))
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty((need,), dtype=torch.uint8, device=self.device)
        return self._ws

    def group_fwd(self, x, tau: float, y=None, routings: list | None = None, stream=None):
        """y: [n_layers, T, d]; routings: one Routing per layer (outputs)."""
        T = x.shape[0]
        n, L0 = len(self.layers), self.layers[0]
        if y is None:
            y = torch.empty((n, T, L0.d), dtype=L0.tdtype, device=self.device)
        if routings is None:
            routings = [l.new_routing(T) for l in self.layers]
        arr = (RoutingStruct * n)(*[r.struct for r in routings])
        ws = self.workspace(T)
        _check(_lib.d2d_group_fwd(self.handle, _ptr(x), T, c_float(tau), _ptr(y), arr, _ptr(ws), ws.numel(),
                                  _stream(stream)), "d2d_group_fwd")
        return y, routings


def select_dynk(R, tau: float, routing: Routing | None = None, dual: bool = False, stream=None,
                perm_capacity: int | None = None) -> Routing:
    T, E = R.shape
    if routing is None:
        routing = Routing(T, E, R.device, dual, perm_capacity)
    nbytes = int(_lib.d2d_select_workspace_bytes(T, E))
    ws = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=R.device)
    _check(_lib.d2d_select_dynk(_ptr(R), T, E, c_float(tau), ctypes.byref(routing.struct), _ptr(ws), ws.numel(),
                                _stream(stream)), "d2d_select_dynk")
    return routing


def select_dynk_static(R, tau: float, routing: Routing, stream=None) -> Routing:
    """d2d_select_dynk_static: selection whose scratch is a fixed array inside the library, for callers that
    may not allocate device memory.  `routing` (the outputs) must be supplied by the caller; nothing is allocated here."""
    T, E = R.shape
    _check(_lib.d2d_select_dynk_static(_ptr(R), T, E, c_float(tau), ctypes.byref(routing.struct), _stream(stream)),
           "d2d_select_dynk_static")
    return routing


def select_topk(R, kk: int, routing: Routing | None = None, dual: bool = False, stream=None) -> Routing:
    T, E = R.shape
    if routing is None:
        routing = Routing(T, E, R.device, dual)
    nbytes = int(_lib.d2d_select_workspace_bytes(T, E))
    ws = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=R.device)
    _check(_lib.d2d_select_topk(_ptr(R), T, E, int(kk), ctypes.byref(routing.struct), _ptr(ws), ws.numel(),
                                _stream(stream)), "d2d_select_topk")
    return routing


def routing_from_mask(mask_words, E: int, dual: bool = False, stream=None) -> Routing:
    """mask_words: device int32 tensor [T, ceil(E/32)] holding the uint32 mask words."""
    T = mask_words.shape[0]
    routing = Routing(T, E, mask_words.device, dual)
    routing.mask.copy_(mask_words)
    nbytes = int(_lib.d2d_select_workspace_bytes(T, E))
    ws = torch.empty((max(nbytes, 256),), dtype=torch.uint8, device=mask_words.device)
    _check(_lib.d2d_routing_from_mask(T, E, ctypes.byref(routing.struct), _ptr(ws), ws.numel(), _stream(stream)),
           "d2d_routing_from_mask")
    return routing


# C-ABI names, for callers that prefer them
d2d_select_dynk = select_dynk
d2d_select_topk = select_topk
d2d_routing_from_mask = routing_from_mask


def d2d_router_fwd(layer: Layer, x, **kw):
    return layer.router_fwd(x, **kw)


def d2d_moe_ffn_fwd(layer: Layer, x, routing: Routing, **kw):
    return layer.moe_ffn_fwd(x, routing, **kw)


def d2d_layer_fwd(layer: Layer, x, tau: float, **kw):
    return layer.layer_fwd(x, tau, **kw)


def to_device(a, dtype_name: str, device="cuda:0"):
    """numpy float32 array (bf16-representable for bf16 layers) -> device tensor of the layer dtype."""
    return torch.from_numpy(a).to(device=device, dtype=torch_dtype(dtype_name)).contiguous()

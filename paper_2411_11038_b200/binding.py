"""ctypes binding of libefqat.so: argument marshalling only.

Function names mirror include/efqat.h and include/efqat_aux.h.  Tensors are torch CUDA tensors used purely as
device memory; every computation happens inside the library's kernels.  Importing this
module does not load the library; the first call does, and fails loudly if the shared
object has not been built (python -m paper_2411_11038_b200.build).
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libefqat.so")

CWPL, CWPN, LWPN = 0, 1, 2
F32, BF16 = 0, 1

EXPORTS = [
    "efqat_create", "efqat_destroy", "efqat_status_string", "efqat_device_status",
    "efqat_ratio_to_k", "efqat_validate_layer", "efqat_workspace_bytes",
    "efqat_select_workspace_bytes", "efqat_select_channels", "efqat_fq_linear_fwd",
    "efqat_fq_linear_bwd", "efqat_fake_quant_act", "efqat_fake_quant_weight",
    "efqat_init_act_qparams", "efqat_init_weight_scales", "efqat_gemm_bf16",
    "efqat_profile_enable", "efqat_profile_read", "efqat_launch_count", "efqat_colsum_noalloc",
    "efqat_selftest_bounded_wait", "efqat_qparam_adam", "efqat_log2_scale_init",
    "efqat_weight_cache_bytes", "efqat_weight_cache_update", "efqat_fq_linear_fwd_cached",
    "efqat_fq_linear_bwd_cached", "efqat_network_fwd", "efqat_network_bwd", "efqat_network_cache_update",
    "efqat_network_qparam_adam",
]


class QSpec(C.Structure):
    _fields_ = [("w_bits", C.c_int), ("x_bits", C.c_int), ("x_symmetric", C.c_int)]


class LayerDesc(C.Structure):
    _fields_ = [("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("is_conv", C.c_int),
                ("B", C.c_int), ("H", C.c_int), ("W", C.c_int), ("Cin", C.c_int), ("R", C.c_int),
                ("S", C.c_int), ("stride", C.c_int), ("pad", C.c_int), ("act_dtype", C.c_int)]


class Sgd(C.Structure):
    _fields_ = [("lr", C.c_float), ("momentum", C.c_float), ("weight_decay", C.c_float),
                ("W_inout", C.c_void_p), ("mom_inout", C.c_void_p)]


class Adam(C.Structure):
    _fields_ = [("lr", C.c_float), ("beta1", C.c_float), ("beta2", C.c_float), ("eps", C.c_float),
                ("step", C.c_int64), ("log2_scale", C.c_int)]


class QParamState(C.Structure):
    _fields_ = [("s_w", C.c_void_p), ("m_sw", C.c_void_p), ("v_sw", C.c_void_p), ("theta_sw", C.c_void_p),
                ("s_x", C.c_void_p), ("z_x", C.c_void_p), ("state_x", C.c_void_p)]


class NetLayer(C.Structure):
    """efqat_net_layer: the arguments of one layer's forward / backward calls, gathered."""
    _fields_ = [("layer", LayerDesc), ("q", QSpec),
                ("X", C.c_void_p), ("W", C.c_void_p), ("s_w", C.c_void_p), ("s_x", C.c_void_p), ("z_x", C.c_void_p),
                ("bias_or_null", C.c_void_p), ("Y", C.c_void_p),
                ("dY", C.c_void_p), ("idx", C.c_void_p), ("k_sel", C.c_int64),
                ("dX", C.c_void_p), ("dW_sel", C.c_void_p), ("dS_w_sel", C.c_void_p), ("dS_x", C.c_void_p),
                ("dZ_x", C.c_void_p), ("db_or_null", C.c_void_p),
                ("opt_or_null", C.POINTER(Sgd)),
                ("cache_or_null", C.c_void_p), ("cache_bytes", C.c_size_t),
                ("ws", C.c_void_p), ("ws_bytes", C.c_size_t)]


class EfqatError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: efqat status {code} ({status_string(code)})")


_lib = None


def load() -> C.CDLL:
    """Loads libefqat.so once.  No fallback: a missing library is an error."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2411_11038_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i64, i32, sz = C.c_void_p, C.c_int64, C.c_int, C.c_size_t
    lib.efqat_create.argtypes = [C.POINTER(vp), i32]
    lib.efqat_destroy.argtypes = [vp]
    lib.efqat_status_string.argtypes = [i32]
    lib.efqat_status_string.restype = C.c_char_p
    lib.efqat_device_status.argtypes = [vp, C.POINTER(i32)]
    lib.efqat_ratio_to_k.argtypes = [C.c_double, i64]
    lib.efqat_ratio_to_k.restype = i64
    lib.efqat_validate_layer.argtypes = [C.POINTER(LayerDesc), C.POINTER(QSpec)]
    lib.efqat_workspace_bytes.argtypes = [C.POINTER(LayerDesc), C.POINTER(QSpec), i64, C.POINTER(sz)]
    lib.efqat_select_workspace_bytes.argtypes = [i32, i64, C.POINTER(sz)]
    lib.efqat_select_channels.argtypes = [vp, i32, i32, C.POINTER(LayerDesc), C.POINTER(vp), C.POINTER(i64),
                                          vp, vp, vp, vp, sz, vp]
    lib.efqat_fq_linear_fwd.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(QSpec), vp, vp, vp, vp, vp, vp, vp,
                                        vp, sz, vp]
    lib.efqat_fq_linear_bwd.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(QSpec), vp, vp, vp, vp, vp, vp,
                                        vp, i64, vp, vp, vp, vp, vp, vp, C.POINTER(Sgd), vp, sz, vp]
    lib.efqat_fake_quant_act.argtypes = [vp, C.POINTER(QSpec), i32, vp, i64, vp, vp, vp, vp, vp]
    lib.efqat_fake_quant_weight.argtypes = [vp, C.POINTER(QSpec), vp, i64, i64, vp, vp, vp, vp]
    lib.efqat_init_act_qparams.argtypes = [vp, C.POINTER(QSpec), i32, vp, i64, vp, vp, vp, sz, vp]
    lib.efqat_init_weight_scales.argtypes = [vp, C.POINTER(QSpec), vp, i64, i64, vp, vp]
    lib.efqat_gemm_bf16.argtypes = [vp, vp, vp, i64, i64, i64, i32, i32, i32, vp, vp]
    lib.efqat_profile_enable.argtypes = [vp, i32]
    lib.efqat_profile_read.argtypes = [vp, i32, C.POINTER(C.c_float), C.POINTER(i32)]
    lib.efqat_colsum_noalloc.argtypes = [i32, vp, i64, i64, vp, vp]
    lib.efqat_launch_count.argtypes = [vp]
    lib.efqat_launch_count.restype = i64
    lib.efqat_selftest_bounded_wait.argtypes = [vp, C.c_uint64, vp]
    lib.efqat_qparam_adam.argtypes = [vp, C.POINTER(Adam), C.POINTER(QParamState), i64, vp, i64, vp, vp, vp, vp]
    lib.efqat_log2_scale_init.argtypes = [vp, vp, vp, i64, vp]
    lib.efqat_weight_cache_bytes.argtypes = [C.POINTER(LayerDesc), C.POINTER(QSpec), C.POINTER(sz)]
    lib.efqat_weight_cache_update.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(QSpec), vp, vp, vp, i64, vp, sz, vp]
    lib.efqat_fq_linear_fwd_cached.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(QSpec), vp, vp, vp, vp, vp, vp,
                                               vp, sz, vp, sz, vp]
    lib.efqat_fq_linear_bwd_cached.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(QSpec), vp, vp, vp, vp, vp, vp,
                                               vp, i64, vp, vp, vp, vp, vp, vp, C.POINTER(Sgd), vp, sz, vp, sz, vp]
    for nm in ("efqat_network_fwd", "efqat_network_bwd", "efqat_network_cache_update"):
        getattr(lib, nm).argtypes = [vp, i32, C.POINTER(NetLayer), vp]
    lib.efqat_network_qparam_adam.argtypes = [vp, C.POINTER(Adam), i32, C.POINTER(NetLayer), C.POINTER(QParamState), vp]
    for name in EXPORTS:
        fn = getattr(lib, name)
        if name not in ("efqat_status_string", "efqat_ratio_to_k", "efqat_launch_count"):
            fn.restype = i32
    _lib = lib
    return lib


def status_string(code: int) -> str:
    return load().efqat_status_string(int(code)).decode()


def _check(rc: int, where: str):
    if rc != 0:
        raise EfqatError(rc, where)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


_raw_stream = getattr(torch._C, "_cuda_getCurrentRawStream", None)


def _stream() -> C.c_void_p:
    """Handle of torch's current CUDA stream on the current device (the raw-handle query is
    ten times cheaper than building a torch.cuda.Stream object, and this runs on every call)."""
    if _raw_stream is not None:
        return C.c_void_p(_raw_stream(torch.cuda.current_device()))
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"activations must be fp32 or bf16, got {t.dtype}")


def _dev(t: torch.Tensor) -> torch.Tensor:
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return t


class Context:
    """efqat_create / efqat_destroy."""

    def __init__(self, device: int = 0):
        lib = load()
        h = C.c_void_p()
        torch.cuda.set_device(device)
        _check(lib.efqat_create(C.byref(h), int(device)), "efqat_create")
        self.handle = h
        self.device = device

    def device_status(self) -> int:
        code = C.c_int(0)
        _check(load().efqat_device_status(self.handle, C.byref(code)), "efqat_device_status")
        return code.value

    def profile_enable(self, on: bool = True):
        _check(load().efqat_profile_enable(self.handle, 1 if on else 0), "efqat_profile_enable")

    def profile_read(self, which: int):
        """(total ms, launches) of kernel `which` (0 fwd, 1 dX, 2 dW GEMM) since the last read."""
        ms, n = C.c_float(0), C.c_int(0)
        _check(load().efqat_profile_read(self.handle, int(which), C.byref(ms), C.byref(n)), "efqat_profile_read")
        return ms.value, n.value

    def launch_count(self) -> int:
        """Kernels launched through this context so far."""
        return int(load().efqat_launch_count(self.handle))

    def selftest_bounded_wait(self, limit_ns: int = 1_000_000):
        """efqat_selftest_bounded_wait: a wait nobody satisfies; read the outcome with device_status()."""
        _check(load().efqat_selftest_bounded_wait(self.handle, int(limit_ns), _stream()),
               "efqat_selftest_bounded_wait")

    def close(self):
        if getattr(self, "handle", None):
            load().efqat_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


@dataclass
class ConvGeom:
    B: int
    H: int
    W: int
    Cin: int
    R: int
    S: int
    stride: int = 1
    pad: int = 0


def layer_desc(M: int, N: int, K: int, act_dtype: int, conv: Optional[ConvGeom] = None) -> LayerDesc:
    d = LayerDesc(M=M, N=N, K=K, is_conv=0, B=1, H=1, W=1, Cin=K, R=1, S=1, stride=1, pad=0,
                  act_dtype=act_dtype)
    if conv is not None:
        d.is_conv = 1
        d.B, d.H, d.W, d.Cin, d.R, d.S, d.stride, d.pad = (conv.B, conv.H, conv.W, conv.Cin, conv.R, conv.S,
                                                         conv.stride, conv.pad)
    return d


def ratio_to_k(ratio: float, n: int) -> int:
    return int(load().efqat_ratio_to_k(float(ratio), int(n)))


def validate_layer(desc: LayerDesc, spec: QSpec) -> int:
    return int(load().efqat_validate_layer(C.byref(desc), C.byref(spec)))


def workspace_bytes(desc: LayerDesc, spec: QSpec, k_sel_max: int) -> int:
    out = C.c_size_t(0)
    _check(load().efqat_workspace_bytes(C.byref(desc), C.byref(spec), int(k_sel_max), C.byref(out)),
           "efqat_workspace_bytes")
    return out.value


def select_workspace_bytes(L: int, total_channels: int) -> int:
    out = C.c_size_t(0)
    _check(load().efqat_select_workspace_bytes(int(L), int(total_channels), C.byref(out)),
           "efqat_select_workspace_bytes")
    return out.value


def weight_cache_bytes(desc: LayerDesc, spec: QSpec) -> int:
    out = C.c_size_t(0)
    _check(load().efqat_weight_cache_bytes(C.byref(desc), C.byref(spec), C.byref(out)), "efqat_weight_cache_bytes")
    return out.value


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


# ---------------------------------------------------------------------------------------
class SelectPlan:
    """Pre-marshalled arguments of efqat_select_channels for a fixed set of layers."""

    def __init__(self, ctx: Context, mode: int, weights: Sequence[torch.Tensor], k: Sequence[int],
                 want_importance: bool = False):
        self.ctx, self.mode = ctx, mode
        self.weights = [_dev(w) for w in weights]
        L = len(weights)
        self.L = L
        self.N = [int(w.shape[0]) for w in weights]
        self.K = [int(w.numel() // w.shape[0]) for w in weights]
        self.total = sum(self.N)
        dev = weights[0].device
        self.descs = (LayerDesc * L)(*[layer_desc(1, n, kk, F32) for n, kk in zip(self.N, self.K)])
        self.wptrs = (C.c_void_p * L)(*[w.data_ptr() for w in self.weights])
        self.k = (C.c_int64 * max(L, 1))(*[int(v) for v in k])
        cap = {CWPL: sum(int(v) for v in k[:L]), CWPN: int(k[0]), LWPN: self.total}[mode]
        self.idx = torch.empty(max(cap, 1), dtype=torch.int32, device=dev)
        self.offsets = torch.empty(L + 1, dtype=torch.int32, device=dev)
        n_imp = L if mode == LWPN else self.total
        self.importance = torch.empty(n_imp, dtype=torch.float32, device=dev) if want_importance else None
        self.ws = alloc_workspace(select_workspace_bytes(L, self.total), dev)

    def run(self):
        rc = load().efqat_select_channels(self.ctx.handle, self.mode, self.L, self.descs, self.wptrs, self.k,
                                          _ptr(self.idx), _ptr(self.offsets), _ptr(self.importance),
                                          _ptr(self.ws), self.ws.numel(), _stream())
        _check(rc, "efqat_select_channels")
        return self.idx, self.offsets, self.importance


def select_channels(ctx: Context, mode: int, weights: Sequence[torch.Tensor], k: Sequence[int],
                    want_importance: bool = False):
    """Returns (list of per-layer int32 index tensors, offsets tensor, importance or None)."""
    plan = SelectPlan(ctx, mode, weights, k, want_importance)
    idx, offsets, imp = plan.run()
    off = offsets.cpu().tolist()
    per_layer = [idx[off[l]:off[l + 1]] for l in range(plan.L)]
    return per_layer, offsets, imp


# ---------------------------------------------------------------------------------------
class LayerPlan:
    """Pre-marshalled forward / backward calls of one layer: descriptor, quantizer spec,
    workspace and output tensors allocated once, so a step is only the two C calls."""

    def __init__(self, ctx: Context, M: int, N: int, K: int, act_dtype: torch.dtype, w_bits: int, x_bits: int,
                 x_symmetric: bool, k_sel_max: int, device, conv: Optional[ConvGeom] = None,
                 x_shape=None, y_shape=None, with_cache: bool = False, ws: Optional[torch.Tensor] = None,
                 outputs: Optional["LayerPlan"] = None):
        """with_cache: also allocate the layer's weight-operand cache (fill it with cache_update).
        ws: a workspace shared with other plans (calls on one stream only).  outputs: another plan
        of the same shape whose output tensors this one reuses (layers timed one after another)."""
        self.ctx = ctx
        self.M, self.N, self.K = M, N, K
        self.act_dtype = act_dtype
        code = F32 if act_dtype == torch.float32 else BF16
        self.desc = layer_desc(M, N, K, code, conv)
        self.spec = QSpec(w_bits, x_bits, 1 if x_symmetric else 0)
        self.k_sel_max = k_sel_max
        self.ws_bytes = workspace_bytes(self.desc, self.spec, k_sel_max)
        if ws is not None and ws.numel() < self.ws_bytes:
            raise ValueError("shared workspace too small for this layer")
        self.ws = ws if ws is not None else alloc_workspace(self.ws_bytes, device)
        xs = tuple(x_shape) if x_shape is not None else (M, K)
        ys = tuple(y_shape) if y_shape is not None else (M, N)
        if outputs is not None:
            if (outputs.M, outputs.N, outputs.K, outputs.act_dtype) != (M, N, K, act_dtype) or \
                    outputs.k_sel_max < k_sel_max:
                raise ValueError("output tensors can only be shared between plans of one shape")
            self.Y, self.dX, self.dW_sel, self.db = outputs.Y, outputs.dX, outputs.dW_sel, outputs.db
        else:
            self.Y = torch.empty(ys, dtype=act_dtype, device=device)
            self.dX = torch.empty(xs, dtype=act_dtype, device=device)
            self.dW_sel = torch.empty((max(k_sel_max, 1), K), dtype=torch.float32, device=device)
            self.db = torch.empty(N, dtype=torch.float32, device=device)
        self.dS_w_sel = torch.empty(max(k_sel_max, 1), dtype=torch.float32, device=device)
        self.dS_x = torch.empty(1, dtype=torch.float32, device=device)
        self.dZ_x = torch.empty(1, dtype=torch.float32, device=device)
        self.cache = alloc_workspace(weight_cache_bytes(self.desc, self.spec), device) if with_cache else None

    def fwd(self, X, W, s_w, s_x, z_x, bias=None):
        rc = load().efqat_fq_linear_fwd(self.ctx.handle, C.byref(self.desc), C.byref(self.spec), _ptr(X), _ptr(W),
                                        _ptr(s_w), _ptr(s_x), _ptr(z_x), _ptr(bias), _ptr(self.Y), _ptr(self.ws),
                                        self.ws.numel(), _stream())
        _check(rc, "efqat_fq_linear_fwd")
        return self.Y

    def bwd(self, dY, X, W, s_w, s_x, z_x, idx, k_sel: int, want_db: bool = True, sgd: Optional[Sgd] = None):
        rc = load().efqat_fq_linear_bwd(self.ctx.handle, C.byref(self.desc), C.byref(self.spec), _ptr(dY), _ptr(X),
                                        _ptr(W), _ptr(s_w), _ptr(s_x), _ptr(z_x), _ptr(idx), int(k_sel),
                                        _ptr(self.dX), _ptr(self.dW_sel), _ptr(self.dS_w_sel), _ptr(self.dS_x),
                                        _ptr(self.dZ_x), _ptr(self.db) if want_db else None,
                                        C.byref(sgd) if sgd is not None else None, _ptr(self.ws),
                                        self.ws.numel(), _stream())
        _check(rc, "efqat_fq_linear_bwd")
        return dict(dX=self.dX, dW_sel=self.dW_sel[:k_sel], dS_w_sel=self.dS_w_sel[:k_sel], dS_x=self.dS_x,
                    dZ_x=self.dZ_x, db=self.db if want_db else None)


    # ---- weight-operand cache ------------------------------------------------------------
    def cache_update(self, W, s_w, idx=None, k_sel: Optional[int] = None):
        """efqat_weight_cache_update: rows idx[0..k_sel) of the cache (default: every row)."""
        k = self.N if k_sel is None else int(k_sel)
        rc = load().efqat_weight_cache_update(self.ctx.handle, C.byref(self.desc), C.byref(self.spec), _ptr(W),
                                              _ptr(s_w), _ptr(idx), k, _ptr(self.cache), self.cache.numel(), _stream())
        _check(rc, "efqat_weight_cache_update")

    def fwd_cached(self, X, s_w, s_x, z_x, bias=None):
        rc = load().efqat_fq_linear_fwd_cached(self.ctx.handle, C.byref(self.desc), C.byref(self.spec), _ptr(X),
                                               _ptr(s_w), _ptr(s_x), _ptr(z_x), _ptr(bias), _ptr(self.Y),
                                               _ptr(self.cache), self.cache.numel(), _ptr(self.ws), self.ws.numel(),
                                               _stream())
        _check(rc, "efqat_fq_linear_fwd_cached")
        return self.Y

    def bwd_cached(self, dY, X, W, s_w, s_x, z_x, idx, k_sel: int, want_db: bool = True, sgd: Optional[Sgd] = None):
        rc = load().efqat_fq_linear_bwd_cached(self.ctx.handle, C.byref(self.desc), C.byref(self.spec), _ptr(dY),
                                               _ptr(X), _ptr(W), _ptr(s_w), _ptr(s_x), _ptr(z_x), _ptr(idx), int(k_sel),
                                               _ptr(self.dX), _ptr(self.dW_sel), _ptr(self.dS_w_sel), _ptr(self.dS_x),
                                               _ptr(self.dZ_x), _ptr(self.db) if want_db else None,
                                               C.byref(sgd) if sgd is not None else None, _ptr(self.cache),
                                               self.cache.numel(), _ptr(self.ws), self.ws.numel(), _stream())
        _check(rc, "efqat_fq_linear_bwd_cached")
        return dict(dX=self.dX, dW_sel=self.dW_sel[:k_sel], dS_w_sel=self.dS_w_sel[:k_sel], dS_x=self.dS_x,
                    dZ_x=self.dZ_x, db=self.db if want_db else None)

    def net_layer(self, X, W, s_w, s_x, z_x, bias, dY, sgd: Optional[Sgd] = None, want_db: bool = True,
                  use_cache: bool = True) -> NetLayer:
        """This layer's entry of an efqat_net_layer array (idx / k_sel are set per step)."""
        n = NetLayer()
        n.layer, n.q = self.desc, self.spec
        n.X, n.W, n.s_w, n.s_x, n.z_x = (t.data_ptr() for t in (X, W, s_w, s_x, z_x))
        n.bias_or_null = bias.data_ptr() if bias is not None else None
        n.Y = self.Y.data_ptr()
        n.dY = dY.data_ptr()
        n.idx, n.k_sel = None, 0
        n.dX, n.dW_sel, n.dS_w_sel = self.dX.data_ptr(), self.dW_sel.data_ptr(), self.dS_w_sel.data_ptr()
        n.dS_x, n.dZ_x = self.dS_x.data_ptr(), self.dZ_x.data_ptr()
        n.db_or_null = self.db.data_ptr() if want_db else None
        n.opt_or_null = C.pointer(sgd) if sgd is not None else None
        if use_cache and self.cache is not None:
            n.cache_or_null, n.cache_bytes = self.cache.data_ptr(), self.cache.numel()
        n.ws, n.ws_bytes = self.ws.data_ptr(), self.ws.numel()
        return n


class NetworkPlan:
    """efqat_network_fwd / _bwd / _cache_update over a fixed list of layers: the efqat_net_layer
    array is marshalled once; a step only rewrites the per-layer (idx, k_sel)."""

    def __init__(self, ctx: Context, entries: Sequence[NetLayer], keep=()):
        self.ctx, self.L = ctx, len(entries)
        self.arr = (NetLayer * self.L)(*entries)
        self.keep = (list(entries), list(keep))     # the structs (and Sgd objects) the pointers refer to

    def set_selection(self, idx: torch.Tensor, offsets_host: Sequence[int]):
        """Per-layer views of the concatenated index list of efqat_select_channels."""
        self.idx = idx
        base, es = idx.data_ptr(), idx.element_size()
        for l in range(self.L):
            k = int(offsets_host[l + 1] - offsets_host[l])
            self.arr[l].k_sel = k
            self.arr[l].idx = (base + es * int(offsets_host[l])) if k else None

    def fwd(self):
        _check(load().efqat_network_fwd(self.ctx.handle, self.L, self.arr, _stream()), "efqat_network_fwd")

    def bwd(self):
        _check(load().efqat_network_bwd(self.ctx.handle, self.L, self.arr, _stream()), "efqat_network_bwd")

    def cache_update(self):
        _check(load().efqat_network_cache_update(self.ctx.handle, self.L, self.arr, _stream()),
               "efqat_network_cache_update")

    def qparam_adam(self, qopts: Sequence["QParamOptimizer"]):
        """efqat_network_qparam_adam: one Adam step on every layer's quantization parameters (the
        optimizers must share their hyper-parameters; their step counters advance together)."""
        if not hasattr(self, "_states"):
            self._states = (QParamState * self.L)(*[q.state for q in qopts])
        for q in qopts:
            q.opt.step += 1
        _check(load().efqat_network_qparam_adam(self.ctx.handle, C.byref(qopts[0].opt), self.L, self.arr, self._states,
                                                _stream()), "efqat_network_qparam_adam")


def _plan_for(ctx, X, W, w_bits, x_bits, x_symmetric, k_sel_max, conv):
    N = int(W.shape[0])
    K = int(W.numel() // N)
    if conv is not None:
        Ho = (conv.H + 2 * conv.pad - conv.R) // conv.stride + 1
        Wo = (conv.W + 2 * conv.pad - conv.S) // conv.stride + 1
        M = conv.B * Ho * Wo
        return LayerPlan(ctx, M, N, K, X.dtype, w_bits, x_bits, x_symmetric, k_sel_max, X.device, conv,
                         x_shape=X.shape, y_shape=(conv.B, Ho, Wo, N))
    M = int(X.shape[0])
    return LayerPlan(ctx, M, N, K, X.dtype, w_bits, x_bits, x_symmetric, k_sel_max, X.device)


def fq_linear_fwd(ctx: Context, X, W, s_w, s_x, z_x, bias=None, w_bits=8, x_bits=8, x_symmetric=False,
                  conv: Optional[ConvGeom] = None):
    """efqat_fq_linear_fwd: returns Y (new tensor)."""
    for t in (X, W, s_w, s_x):
        _dev(t)
    plan = _plan_for(ctx, X, W, w_bits, x_bits, x_symmetric, 0, conv)
    return plan.fwd(X, W, s_w, s_x, z_x, bias)


def fq_linear_bwd(ctx: Context, dY, X, W, s_w, s_x, z_x, idx, k_sel: int, w_bits=8, x_bits=8,
                  x_symmetric=False, want_db=True, sgd: Optional[Sgd] = None, conv: Optional[ConvGeom] = None):
    """efqat_fq_linear_bwd: returns dict(dX, dW_sel, dS_w_sel, dS_x, dZ_x, db)."""
    for t in (dY, X, W, s_w, s_x):
        _dev(t)
    plan = _plan_for(ctx, X, W, w_bits, x_bits, x_symmetric, int(k_sel), conv)
    return plan.bwd(dY, X, W, s_w, s_x, z_x, idx, int(k_sel), want_db, sgd)


def make_sgd(lr: float, momentum: float, weight_decay: float, W: torch.Tensor, mom: torch.Tensor) -> Sgd:
    return Sgd(lr, momentum, weight_decay, W.data_ptr(), mom.data_ptr())


# ---------------------------------------------------------------------------------------
class QParamOptimizer:
    """efqat_qparam_adam for one layer: owns the Adam moments (and theta = log2 s in log2 mode) of
    the layer's weight scales, activation scale and activation zero point."""

    def __init__(self, ctx: Context, s_w, s_x, z_x, lr: float, beta1=0.9, beta2=0.999, eps=1e-8,
                 log2_scale: bool = False):
        self.ctx, self.s_w, self.s_x, self.z_x = ctx, _dev(s_w), _dev(s_x), z_x
        self.N = int(s_w.numel())
        dev = s_w.device
        self.m_sw = torch.zeros(self.N, dtype=torch.float32, device=dev)
        self.v_sw = torch.zeros(self.N, dtype=torch.float32, device=dev)
        self.theta_sw = torch.zeros(self.N, dtype=torch.float32, device=dev) if log2_scale else None
        self.state_x = torch.zeros(8, dtype=torch.float32, device=dev)
        self.opt = Adam(lr, beta1, beta2, eps, 0, 1 if log2_scale else 0)
        if log2_scale:
            lib = load()
            _check(lib.efqat_log2_scale_init(ctx.handle, _ptr(s_w), _ptr(self.theta_sw), self.N, _stream()),
                   "efqat_log2_scale_init")
            _check(lib.efqat_log2_scale_init(ctx.handle, _ptr(s_x), C.c_void_p(self.state_x.data_ptr() + 16), 1,
                                             _stream()), "efqat_log2_scale_init")
        self.state = QParamState(_ptr(s_w), _ptr(self.m_sw), _ptr(self.v_sw), _ptr(self.theta_sw), _ptr(s_x),
                                 _ptr(z_x), _ptr(self.state_x))

    def step(self, idx, k_sel: int, dS_w_sel, dS_x, dZ_x=None):
        self.opt.step += 1
        rc = load().efqat_qparam_adam(self.ctx.handle, C.byref(self.opt), C.byref(self.state), self.N, _ptr(idx),
                                      int(k_sel), _ptr(dS_w_sel), _ptr(dS_x), _ptr(dZ_x), _stream())
        _check(rc, "efqat_qparam_adam")


def fake_quant_act(ctx: Context, x, s_x, z_x, x_bits=8, x_symmetric=False):
    """efqat_fake_quant_act: returns (codes int32, clip uint8) shaped like x."""
    _dev(x)
    spec = QSpec(8, x_bits, 1 if x_symmetric else 0)
    codes = torch.empty(x.shape, dtype=torch.int32, device=x.device)
    clip = torch.empty(x.shape, dtype=torch.uint8, device=x.device)
    rc = load().efqat_fake_quant_act(ctx.handle, C.byref(spec), _dtype_code(x), _ptr(x), x.numel(), _ptr(s_x),
                                     _ptr(z_x), _ptr(codes), _ptr(clip), _stream())
    _check(rc, "efqat_fake_quant_act")
    return codes, clip


def fake_quant_weight(ctx: Context, W, s_w, w_bits=8):
    """efqat_fake_quant_weight: returns (codes int32, clip uint8) shaped like W."""
    _dev(W)
    spec = QSpec(w_bits, 8, 0)
    N = int(W.shape[0])
    K = int(W.numel() // N)
    codes = torch.empty(W.shape, dtype=torch.int32, device=W.device)
    clip = torch.empty(W.shape, dtype=torch.uint8, device=W.device)
    rc = load().efqat_fake_quant_weight(ctx.handle, C.byref(spec), _ptr(W), N, K, _ptr(s_w), _ptr(codes),
                                        _ptr(clip), _stream())
    _check(rc, "efqat_fake_quant_weight")
    return codes, clip


def init_act_qparams(ctx: Context, x, x_bits=8, x_symmetric=False):
    """efqat_init_act_qparams: returns (s_x[1], z_x[1])."""
    _dev(x)
    spec = QSpec(8, x_bits, 1 if x_symmetric else 0)
    s = torch.empty(1, dtype=torch.float32, device=x.device)
    z = torch.empty(1, dtype=torch.float32, device=x.device)
    ws = alloc_workspace(8192, x.device)
    rc = load().efqat_init_act_qparams(ctx.handle, C.byref(spec), _dtype_code(x), _ptr(x), x.numel(), _ptr(s),
                                       _ptr(z), _ptr(ws), ws.numel(), _stream())
    _check(rc, "efqat_init_act_qparams")
    return s, z


def init_weight_scales(ctx: Context, W, w_bits=8):
    """efqat_init_weight_scales: returns s_w[N]."""
    _dev(W)
    spec = QSpec(w_bits, 8, 0)
    N = int(W.shape[0])
    K = int(W.numel() // N)
    s = torch.empty(N, dtype=torch.float32, device=W.device)
    rc = load().efqat_init_weight_scales(ctx.handle, C.byref(spec), _ptr(W), N, K, _ptr(s), _stream())
    _check(rc, "efqat_init_weight_scales")
    return s


def gemm_bf16(ctx: Context, A, B, M: int, N: int, K: int, a_mn: bool, b_mn: bool, splits: int = 1):
    """efqat_gemm_bf16: returns the fp32 slabs [splits, N, M] (transposed product per split)."""
    _dev(A)
    _dev(B)
    out = torch.empty((splits, N, M), dtype=torch.float32, device=A.device)
    rc = load().efqat_gemm_bf16(ctx.handle, _ptr(A), _ptr(B), M, N, K, int(a_mn), int(b_mn), int(splits),
                                _ptr(out), _stream())
    _check(rc, "efqat_gemm_bf16")
    return out


def colsum_noalloc(dY: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """efqat_colsum_noalloc: column sums of a 2-D dY without context or workspace.  The
    library call allocates nothing; `out` (fp32 [N]) is created here only if not given."""
    _dev(dY)
    M, N = int(dY.shape[0]), int(dY.shape[1])
    if out is None:
        out = torch.empty(N, dtype=torch.float32, device=dY.device)
    rc = load().efqat_colsum_noalloc(_dtype_code(dY), _ptr(dY), M, N, _ptr(out), _stream())
    _check(rc, "efqat_colsum_noalloc")
    return out

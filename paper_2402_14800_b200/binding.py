"""Thin ctypes binding of ``libmoe.so`` (see ``include/moe.h``).

Argument marshalling only: every step of the path runs in the library's CUDA
kernels.  Tensors are ``torch`` CUDA tensors used as device memory; the
library is given their ``data_ptr()``.  There is no CPU fallback: if the
library is missing or a call fails, a ``MoeError`` is raised.
"""
from __future__ import annotations

import ctypes
import os
from math import comb

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG, "libmoe.so")

MOE_OK = 0
STATUS_NAMES = {
    0: "MOE_OK", -1: "MOE_ERR_INVALID_ARG", -2: "MOE_ERR_UNSUPPORTED_SHAPE", -3: "MOE_ERR_CUDA",
    -4: "MOE_ERR_OOM", -5: "MOE_ERR_DEVICE_TIMEOUT", -6: "MOE_ERR_ARCH",
}


class MoeError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__("%s: %s" % (STATUS_NAMES.get(code, str(code)), message))
        self.code = code


_lib = None


def load_library(path: str | None = None):
    """Load ``libmoe.so`` (built by ``python -m paper_2402_14800_b200.build``)."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    p = path or _LIB_PATH
    if not os.path.exists(p):
        raise MoeError(-3, "%s not found: build it with `python -m paper_2402_14800_b200.build`" % p)
    lib = ctypes.CDLL(p)
    vp, ci, cf, u32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_uint32
    lib.moe_layer_create.restype = vp
    lib.moe_layer_create.argtypes = [vp, vp, vp, vp, ci, ci, ci, u32]
    lib.moe_layer_destroy.restype = None
    lib.moe_layer_destroy.argtypes = [vp]
    lib.moe_set_stream.argtypes = [vp, vp]
    lib.moe_layer_weight_bytes.restype = ctypes.c_size_t
    lib.moe_layer_weight_bytes.argtypes = [vp]
    lib.moe_layer_scratch_bytes.restype = ctypes.c_size_t
    lib.moe_layer_scratch_bytes.argtypes = [vp]
    lib.moe_forward.argtypes = [vp, vp, ci, cf, vp, vp]
    lib.moe_forward_residual.argtypes = [vp, vp, ci, cf, vp, vp, vp]
    lib.moe_forward_host.argtypes = [vp, vp, ci, cf, vp]
    lib.moe_top2_distance.argtypes = [vp, vp, ci, vp]
    lib.moe_forward_topk.argtypes = [vp, vp, ci, ci, cf, vp, vp, vp, vp]
    lib.moe_routing_stats_layout.restype = ctypes.c_size_t
    lib.moe_routing_stats_layout.argtypes = [ci, ci, ctypes.POINTER(ctypes.c_size_t)]
    lib.moe_routing_stats_bytes.restype = ctypes.c_size_t
    lib.moe_routing_stats_bytes.argtypes = [ci, ci]
    lib.moe_calibrate_beta.argtypes = [vp, vp, ci, ctypes.POINTER(cf)]
    lib.moe_prune_search.argtypes = [vp, vp, ci, ci, ctypes.POINTER(cf), ctypes.POINTER(u32)]
    lib.moe_prune_search_multi.argtypes = [vp, vp, ci, ctypes.POINTER(ci), ci, ctypes.POINTER(cf),
                                           ctypes.POINTER(u32)]
    lib.moe_prune_search_progressive.argtypes = [vp, vp, vp, ci, ci, ctypes.POINTER(cf), ctypes.POINTER(u32)]
    lib.moe_num_subsets.restype = ctypes.c_long
    lib.moe_num_subsets.argtypes = [ci, ci]
    lib.moe_rmsnorm.argtypes = [vp, ci, ci, cf, vp, vp]
    lib.moe_stack_forward.argtypes = [ctypes.POINTER(vp), ci, vp, ci, ctypes.POINTER(cf), cf, vp]
    lib.moe_coselection.argtypes = [vp, vp, ci, ctypes.POINTER(ctypes.c_int32)]
    lib.moe_frequency_subset.restype = u32
    lib.moe_frequency_subset.argtypes = [ctypes.POINTER(ctypes.c_int32), ci, ci]
    lib.moe_device_status.argtypes = [vp]
    lib.moe_layer_share_scratch.argtypes = [vp, vp]
    lib.moe_profile_enable.argtypes = [vp, ci]
    lib.moe_profile_read.argtypes = [vp, ctypes.POINTER(cf), ctypes.POINTER(ci)]
    lib.moe_calibrate_beta_noalloc.argtypes = [vp, vp, ci, ci, ci, vp, ctypes.POINTER(cf)]
    lib.moe_reserve.argtypes = [vp, ci]
    lib.moe_test_wait_expiry.argtypes = [vp, ctypes.c_uint, ci]
    lib.moe_test_set_free_bytes_limit.restype = None
    lib.moe_test_set_free_bytes_limit.argtypes = [ctypes.c_longlong]
    lib.moe_last_error.restype = ctypes.c_char_p
    if path is None:
        _lib = lib
    return lib


def last_error() -> str:
    return load_library().moe_last_error().decode()


def _check(rc: int):
    if rc != MOE_OK:
        raise MoeError(rc, last_error())


def _dev_bf16(t: torch.Tensor, shape=None) -> torch.Tensor:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise MoeError(-1, "expected a contiguous bf16 CUDA tensor")
    if shape is not None and tuple(t.shape) != tuple(shape):
        raise MoeError(-1, "shape %s, expected %s" % (tuple(t.shape), tuple(shape)))
    return t


def routing_stats_layout(T: int, E: int):
    offs = (ctypes.c_size_t * 7)()
    total = load_library().moe_routing_stats_layout(T, E, offs)
    return int(total), [int(o) for o in offs]


def num_subsets(E: int, r: int) -> int:
    return int(load_library().moe_num_subsets(E, r))


class RoutingStats:
    """Device buffer for the routing record of one ``moe_forward`` call, with typed views."""

    def __init__(self, T: int, E: int, device):
        self.T, self.E = T, E
        total, o = routing_stats_layout(T, E)
        self.buf = torch.zeros(max(total, 16), dtype=torch.uint8, device=device)
        b = self.buf
        self.idx = b[o[0]:o[0] + T * 8].view(torch.int32).view(T, 2)
        self.wn = b[o[1]:o[1] + T * 8].view(torch.float32).view(T, 2)
        self.ratio = b[o[2]:o[2] + T * 4].view(torch.float32)
        self.skipped = b[o[3]:o[3] + T]
        self.count = b[o[4]:o[4] + E * 8].view(torch.int32).view(E, 2)
        self.n_skipped = b[o[5]:o[5] + 4].view(torch.int32)
        self.n_experts_touched = b[o[6]:o[6] + 4].view(torch.int32)


class MoeLayer:
    """One MoE layer restricted to the experts of ``kept_mask`` (``moe_layer_create``)."""

    def __init__(self, W_gate, W1, W3, W2, kept_mask: int | None = None):
        lib = load_library()
        E, h = W_gate.shape
        f = W1.shape[1]
        _dev_bf16(W_gate, (E, h)); _dev_bf16(W1, (E, f, h)); _dev_bf16(W3, (E, f, h)); _dev_bf16(W2, (E, h, f))
        self.h, self.f, self.E = h, f, E
        self.kept_mask = (1 << E) - 1 if kept_mask is None else int(kept_mask)
        self.device = W_gate.device
        with torch.cuda.device(self.device):
            self._h = lib.moe_layer_create(W_gate.data_ptr(), W1.data_ptr(), W3.data_ptr(), W2.data_ptr(),
                                           h, f, E, self.kept_mask)
        if not self._h:
            raise MoeError(-1, last_error())
        self.set_stream(torch.cuda.current_stream(self.device))

    def close(self):
        if getattr(self, "_h", None):
            load_library().moe_layer_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_stream(self, stream: torch.cuda.Stream):
        _check(load_library().moe_set_stream(self._h, ctypes.c_void_p(stream.cuda_stream)))

    def share_scratch(self, owner: "MoeLayer | None"):
        """Run out of ``owner``'s scratch buffers (``moe_layer_share_scratch``)."""
        _check(load_library().moe_layer_share_scratch(self._h, owner._h if owner is not None else None))

    def reserve(self, T_max: int):
        """``moe_reserve``: grow the scratch for any forward batch of up to ``T_max`` tokens now."""
        _check(load_library().moe_reserve(self._h, int(T_max)))

    @property
    def weight_bytes(self) -> int:
        return int(load_library().moe_layer_weight_bytes(self._h))

    @property
    def scratch_bytes(self) -> int:
        return int(load_library().moe_layer_scratch_bytes(self._h))

    def forward(self, x, beta: float = 0.0, y=None, stats: RoutingStats | None = None, residual=None):
        """``moe_forward`` / ``moe_forward_residual``; returns y."""
        T = x.shape[0]
        _dev_bf16(x, (T, self.h))
        if y is None:
            y = torch.empty_like(x)
        _dev_bf16(y, (T, self.h))
        sp = stats.buf.data_ptr() if stats is not None else None
        lib = load_library()
        if residual is None:
            _check(lib.moe_forward(self._h, x.data_ptr(), T, beta, y.data_ptr(), sp))
        else:
            _dev_bf16(residual, (T, self.h))
            _check(lib.moe_forward_residual(self._h, x.data_ptr(), T, beta, residual.data_ptr(),
                                            y.data_ptr(), sp))
        return y

    def forward_topk(self, x, k: int, beta: float = 0.0, y=None, record: bool = False):
        """``moe_forward_topk``; with ``record`` also returns (idx[T,k] i32, wn[T,k] f32, n_active[T] i32)."""
        T = x.shape[0]
        _dev_bf16(x, (T, self.h))
        if y is None:
            y = torch.empty_like(x)
        idx = wn = na = None
        if record:
            idx = torch.zeros((T, max(k, 1)), dtype=torch.int32, device=x.device)
            wn = torch.zeros((T, max(k, 1)), dtype=torch.float32, device=x.device)
            na = torch.zeros((T,), dtype=torch.int32, device=x.device)
        _check(load_library().moe_forward_topk(
            self._h, x.data_ptr(), T, k, beta, y.data_ptr(),
            idx.data_ptr() if record else None, wn.data_ptr() if record else None,
            na.data_ptr() if record else None))
        return (y, idx, wn, na) if record else y

    def top2_distance(self, x):
        """``moe_top2_distance``: fp32 CUDA tensor [T] of ||E_e0(x) - E_e1(x)||_2."""
        T = x.shape[0]
        _dev_bf16(x, (T, self.h))
        out = torch.empty((T,), dtype=torch.float32, device=x.device)
        _check(load_library().moe_top2_distance(self._h, x.data_ptr(), T, out.data_ptr()))
        return out

    def forward_host(self, x_host: torch.Tensor, beta: float, y_host: torch.Tensor):
        """``moe_forward_host``: x_host, y_host are host bf16 tensors (pinned or not)."""
        T = x_host.shape[0]
        assert x_host.dtype == torch.bfloat16 and y_host.dtype == torch.bfloat16
        assert not x_host.is_cuda and not y_host.is_cuda and x_host.is_contiguous() and y_host.is_contiguous()
        _check(load_library().moe_forward_host(self._h, x_host.data_ptr(), T, beta, y_host.data_ptr()))
        return y_host

    def calibrate_beta(self, x) -> float:
        T = x.shape[0]
        _dev_bf16(x, (T, self.h))
        out = ctypes.c_float(0)
        _check(load_library().moe_calibrate_beta(self._h, x.data_ptr(), T, ctypes.byref(out)))
        return float(out.value)

    def prune_search(self, x_calib, r: int):
        """``moe_prune_search``; returns (losses list of C(E, r) floats, best_subset bitmask)."""
        T = x_calib.shape[0]
        _dev_bf16(x_calib, (T, self.h))
        n = comb(self.E, r) if 0 <= r <= self.E else 1
        losses = (ctypes.c_float * max(n, 1))()
        best = ctypes.c_uint32(0)
        _check(load_library().moe_prune_search(self._h, x_calib.data_ptr(), T, r, losses, ctypes.byref(best)))
        return list(losses)[:n], int(best.value)

    def prune_search_multi(self, x_calib, rs):
        """``moe_prune_search_multi``: one evaluation of the experts, one enumeration per subset
        size in ``rs``; returns a list of (losses, best_subset) in the order of ``rs``."""
        T = x_calib.shape[0]
        _dev_bf16(x_calib, (T, self.h))
        rs = [int(r) for r in rs]
        ns = [comb(self.E, r) if 0 <= r <= self.E else 1 for r in rs]
        losses = (ctypes.c_float * max(sum(ns), 1))()
        best = (ctypes.c_uint32 * max(len(rs), 1))()
        r_arr = (ctypes.c_int * max(len(rs), 1))(*rs)
        _check(load_library().moe_prune_search_multi(self._h, x_calib.data_ptr(), T, r_arr, len(rs),
                                                     losses, best))
        out, o = [], 0
        for i, n in enumerate(ns):
            out.append((list(losses[o:o + n]), int(best[i])))
            o += n
        return out

    def coselection(self, x):
        """``moe_coselection``: E x E list of lists, counts[a][b] = tokens with top-2 (a, b)."""
        T = x.shape[0]
        _dev_bf16(x, (T, self.h))
        buf = (ctypes.c_int32 * (self.E * self.E))()
        _check(load_library().moe_coselection(self._h, x.data_ptr(), T, buf))
        return [[int(buf[a * self.E + b]) for b in range(self.E)] for a in range(self.E)]

    def frequency_subset(self, counts, r: int) -> int:
        """``moe_frequency_subset``: the activation-frequency baseline's kept mask."""
        flat = [int(v) for row in counts for v in row]
        buf = (ctypes.c_int32 * len(flat))(*flat)
        return int(load_library().moe_frequency_subset(buf, self.E, r))

    def profile_enable(self, on: bool = True):
        _check(load_library().moe_profile_enable(self._h, int(bool(on))))

    def profile_read(self):
        """Returns (stage_ms[4] summed over the recorded calls, number of calls)."""
        ms = (ctypes.c_float * 4)()
        n = ctypes.c_int(0)
        _check(load_library().moe_profile_read(self._h, ms, ctypes.byref(n)))
        return [float(v) for v in ms], int(n.value)

    def prune_search_progressive(self, x_pruned, F_ref, r: int):
        """``moe_prune_search_progressive``: F_ref is a contiguous fp32 CUDA tensor [T, h]."""
        T = x_pruned.shape[0]
        _dev_bf16(x_pruned, (T, self.h))
        if not (F_ref.is_cuda and F_ref.dtype == torch.float32 and F_ref.is_contiguous()
                and tuple(F_ref.shape) == (T, self.h)):
            raise MoeError(-1, "F_ref must be a contiguous fp32 CUDA tensor of shape [T, h]")
        n = comb(self.E, r) if 0 <= r <= self.E else 1
        losses = (ctypes.c_float * max(n, 1))()
        best = ctypes.c_uint32(0)
        _check(load_library().moe_prune_search_progressive(self._h, x_pruned.data_ptr(), F_ref.data_ptr(),
                                                           T, r, losses, ctypes.byref(best)))
        return list(losses)[:n], int(best.value)

    def device_status(self) -> int:
        return int(load_library().moe_device_status(self._h))


def calibrate_beta_noalloc(W_gate_kept, x, stream=None) -> float:
    """``moe_calibrate_beta_noalloc``: the beta median without any device allocation by the
    library (scratch is a fixed array inside it; at most 16384 tokens).  ``W_gate_kept`` holds
    the router rows of the kept experts, ``x`` the calibration tokens."""
    r, h = W_gate_kept.shape
    T = x.shape[0]
    _dev_bf16(W_gate_kept)
    _dev_bf16(x, (T, h))
    st = stream or torch.cuda.current_stream(x.device)
    out = ctypes.c_float(0)
    _check(load_library().moe_calibrate_beta_noalloc(W_gate_kept.data_ptr(), x.data_ptr(), T, h, r,
                                                     ctypes.c_void_p(st.cuda_stream), ctypes.byref(out)))
    return float(out.value)


def rmsnorm(x, eps: float = 1e-5, out=None, stream=None):
    T, h = x.shape
    _dev_bf16(x)
    if out is None:
        out = torch.empty_like(x)
    st = stream or torch.cuda.current_stream(x.device)
    _check(load_library().moe_rmsnorm(x.data_ptr(), T, h, eps, out.data_ptr(), ctypes.c_void_p(st.cuda_stream)))
    return out


def stack_forward(layers, x, betas=None, eps: float = 1e-5, y=None):
    """``moe_stack_forward``: x_{l+1} = x_l + MoE_l(RMSNorm(x_l)) over ``layers``."""
    T, h = x.shape
    _dev_bf16(x)
    if y is None:
        y = torch.empty_like(x)
    n = len(layers)
    arr = (ctypes.c_void_p * n)(*[l._h for l in layers])
    b = None
    if betas is not None:
        b = (ctypes.c_float * n)(*[float(v) for v in betas])
    _check(load_library().moe_stack_forward(arr, n, x.data_ptr(), T, b, eps, y.data_ptr()))
    return y

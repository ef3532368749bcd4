"""ctypes front end of the CPU oracle (``moe_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA path never imports this module, and
this module imports nothing from the CUDA package.

Arguments are numpy arrays; bf16 tensors are ``uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from math import comb

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "moe_oracle.c")
_LIB = os.path.join(_HERE, "libmoe_oracle.so")

_u16p = ctypes.POINTER(ctypes.c_uint16)
_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)
_i32p = ctypes.POINTER(ctypes.c_int32)
_i64p = ctypes.POINTER(ctypes.c_int64)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_u32p = ctypes.POINTER(ctypes.c_uint32)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP, no fast-math)."""
    def stale():
        return force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)

    if stale():
        import fcntl
        with open(_LIB + ".lock", "w") as lock:
            fcntl.flock(lock, fcntl.LOCK_EX)
            if stale():
                tmp = _LIB + ".tmp%d" % os.getpid()
                subprocess.check_call(
                    ["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"]
                )
                os.replace(tmp, _LIB)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_bf16_to_f32.restype = ctypes.c_float
        _lib.oracle_bf16_to_f32.argtypes = [ctypes.c_uint16]
        _lib.oracle_f32_to_bf16.restype = ctypes.c_uint16
        _lib.oracle_f32_to_bf16.argtypes = [ctypes.c_float]
        _lib.oracle_num_subsets.restype = ctypes.c_long
    return _lib


def _p(a, typ):
    return None if a is None else a.ctypes.data_as(typ)


def _u16(a, shape=None):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, "bf16 tensors are passed as uint16 bit patterns"
    if shape is not None:
        assert tuple(a.shape) == tuple(shape), (a.shape, shape)
    return a


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def f32_to_bf16(v: float) -> int:
    return int(lib().oracle_f32_to_bf16(ctypes.c_float(v)))


def bf16_to_f32(b: int) -> float:
    return float(lib().oracle_bf16_to_f32(ctypes.c_uint16(b)))


def enumerate_subsets(E: int, r: int) -> np.ndarray:
    masks = np.zeros(comb(E, r), dtype=np.uint32)
    rc = lib().oracle_enumerate_subsets(E, r, _p(masks, _u32p))
    if rc:
        raise ValueError("bad (E, r)")
    return masks


def route(x, Wg, kept_mask: int, beta: float):
    """Routing of every token among the kept experts.  Returns a dict with
    logits[T,E] f32, idx[T,2] i32, w[T,2], wn[T,2], ratio[T] f32, skipped[T] u8."""
    x = _u16(x)
    T, h = x.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    out = dict(
        logits=np.zeros((T, E), np.float32),
        idx=np.zeros((T, 2), np.int32),
        w=np.zeros((T, 2), np.float32),
        wn=np.zeros((T, 2), np.float32),
        ratio=np.zeros((T,), np.float32),
        skipped=np.zeros((T,), np.uint8),
    )
    rc = lib().oracle_route(
        _p(x, _u16p), _p(Wg, _u16p), T, h, E, ctypes.c_uint32(kept_mask), ctypes.c_float(beta),
        _p(out["logits"], _f32p), _p(out["idx"], _i32p), _p(out["w"], _f32p), _p(out["wn"], _f32p),
        _p(out["ratio"], _f32p), _p(out["skipped"], _u8p))
    if rc:
        raise ValueError("oracle_route: invalid arguments")
    return out


def all_experts(x, W1, W3, W2, round_bf16: bool, expert_mask: int | None = None) -> np.ndarray:
    """Yall[T,E,h] float64: every expert on every token."""
    x = _u16(x)
    T, h = x.shape
    W1 = _u16(W1)
    E, f, _ = W1.shape
    W3 = _u16(W3, (E, f, h))
    W2 = _u16(W2, (E, h, f))
    Y = np.zeros((T, E, h), np.float64)
    m = (1 << E) - 1 if expert_mask is None else expert_mask
    rc = lib().oracle_all_experts(_p(x, _u16p), _p(W1, _u16p), _p(W3, _u16p), _p(W2, _u16p),
                                  T, h, f, E, ctypes.c_uint32(m), int(bool(round_bf16)), _p(Y, _f64p))
    if rc:
        raise ValueError("oracle_all_experts: invalid arguments")
    return Y


def moe_forward(x, Wg, W1, W3, W2, kept_mask: int, beta: float, residual=None):
    """Pruned + skipping layer forward.  Returns dict(y[T,h] u16, z[T,h] f64,
    idx, wn, ratio, skipped)."""
    x = _u16(x)
    T, h = x.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    W1 = _u16(W1)
    f = W1.shape[1]
    W3 = _u16(W3, (E, f, h))
    W2 = _u16(W2, (E, h, f))
    res = None if residual is None else _u16(residual, (T, h))
    out = dict(
        y=np.zeros((T, h), np.uint16),
        z=np.zeros((T, h), np.float64),
        idx=np.zeros((T, 2), np.int32),
        wn=np.zeros((T, 2), np.float32),
        ratio=np.zeros((T,), np.float32),
        skipped=np.zeros((T,), np.uint8),
    )
    rc = lib().oracle_moe_forward(
        _p(x, _u16p), _p(Wg, _u16p), _p(W1, _u16p), _p(W3, _u16p), _p(W2, _u16p), T, h, f, E,
        ctypes.c_uint32(kept_mask), ctypes.c_float(beta), _p(res, _u16p), _p(out["y"], _u16p),
        _p(out["z"], _f64p), _p(out["idx"], _i32p), _p(out["wn"], _f32p), _p(out["ratio"], _f32p),
        _p(out["skipped"], _u8p))
    if rc:
        raise ValueError("oracle_moe_forward: invalid arguments")
    return out


def coselection(x, Wg) -> np.ndarray:
    """counts[E,E] int64: tokens with top-1 expert a and top-2 expert b."""
    x = _u16(x)
    T, h = x.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    counts = np.zeros((E, E), np.int64)
    if lib().oracle_coselection(_p(x, _u16p), _p(Wg, _u16p), T, h, E, _p(counts, _i64p)):
        raise ValueError("oracle_coselection: invalid arguments")
    return counts


def frequency_subset(counts, r: int) -> int:
    counts = np.ascontiguousarray(counts, dtype=np.int64)
    E = counts.shape[0]
    fn = lib().oracle_frequency_subset
    fn.restype = ctypes.c_uint32
    return int(fn(_p(counts, _i64p), E, r))


def top2_distance(x, Wg, W1, W3, W2, kept_mask: int) -> np.ndarray:
    """dist[T] float64: ||E_e0(x) - E_e1(x)||_2 over each token's two selected experts."""
    x = _u16(x)
    T, h = x.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    W1 = _u16(W1)
    f = W1.shape[1]
    W3 = _u16(W3, (E, f, h))
    W2 = _u16(W2, (E, h, f))
    dist = np.zeros(T, np.float64)
    rc = lib().oracle_top2_distance(_p(x, _u16p), _p(Wg, _u16p), _p(W1, _u16p), _p(W3, _u16p),
                                    _p(W2, _u16p), T, h, f, E, ctypes.c_uint32(kept_mask), _p(dist, _f64p))
    if rc:
        raise ValueError("oracle_top2_distance: invalid arguments")
    return dist


def moe_forward_topk(x, Wg, W1, W3, W2, kept_mask: int, k: int, beta: float):
    """Top-k layer forward with the generalised skipping rule.  Returns dict(y, z, idx[T,k],
    wn[T,k], n_active[T], tail_frac[T], logits[T,E])."""
    x = _u16(x)
    T, h = x.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    W1 = _u16(W1)
    f = W1.shape[1]
    W3 = _u16(W3, (E, f, h))
    W2 = _u16(W2, (E, h, f))
    out = dict(
        y=np.zeros((T, h), np.uint16), z=np.zeros((T, h), np.float64),
        idx=np.zeros((T, k), np.int32), wn=np.zeros((T, k), np.float32),
        n_active=np.zeros((T,), np.int32), tail_frac=np.zeros((T,), np.float32),
        logits=np.zeros((T, E), np.float32),
    )
    rc = lib().oracle_moe_forward_topk(
        _p(x, _u16p), _p(Wg, _u16p), _p(W1, _u16p), _p(W3, _u16p), _p(W2, _u16p), T, h, f, E,
        ctypes.c_uint32(kept_mask), k, ctypes.c_float(beta), _p(out["y"], _u16p), _p(out["z"], _f64p),
        _p(out["idx"], _i32p), _p(out["wn"], _f32p), _p(out["n_active"], _i32p),
        _p(out["tail_frac"], _f32p), _p(out["logits"], _f32p))
    if rc:
        raise ValueError("oracle_moe_forward_topk: invalid arguments")
    return out


def beta_median(ratio) -> float:
    ratio = np.ascontiguousarray(ratio, dtype=np.float32)
    b = ctypes.c_float(0)
    rc = lib().oracle_beta_median(_p(ratio, _f32p), int(ratio.shape[0]), ctypes.byref(b))
    if rc:
        raise ValueError("oracle_beta_median: empty input")
    return float(b.value)


def _search(fn, x, Wg, W1, W3, W2, r):
    x = _u16(x)
    T, h = x.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    W1 = _u16(W1)
    f = W1.shape[1]
    W3 = _u16(W3, (E, f, h))
    W2 = _u16(W2, (E, h, f))
    nC = comb(E, r)
    losses = np.zeros(nC, np.float64)
    loss_sq = np.zeros(nC, np.float64)
    n_changed = np.zeros(nC, np.int64)
    best = ctypes.c_uint32(0)
    rc = fn(_p(x, _u16p), _p(Wg, _u16p), _p(W1, _u16p), _p(W3, _u16p), _p(W2, _u16p), T, h, f, E, r,
            _p(losses, _f64p), _p(loss_sq, _f64p), _p(n_changed, _i64p), ctypes.byref(best))
    if rc:
        raise ValueError("oracle search: invalid arguments")
    return dict(losses=losses, loss_sq=loss_sq, n_changed=n_changed, best_subset=int(best.value),
                subsets=enumerate_subsets(E, r))


def prune_search_bruteforce(x, Wg, W1, W3, W2, r: int):
    """Eq. 3 literally: every subset re-runs the pruned layer."""
    return _search(lib().oracle_prune_search_bruteforce, x, Wg, W1, W3, W2, r)


def prune_search_allexperts(x, Wg, W1, W3, W2, r: int):
    """Eq. 3 with the experts evaluated once and gathered per subset."""
    return _search(lib().oracle_prune_search_allexperts, x, Wg, W1, W3, W2, r)


def prune_search_progressive(x_p, Wg, W1, W3, W2, F_ref, r: int):
    """Progressive search: the pruned layer runs on x_p, the target is the cached F_ref[T,h] f32."""
    x_p = _u16(x_p)
    T, h = x_p.shape
    Wg = _u16(Wg)
    E = Wg.shape[0]
    W1 = _u16(W1)
    f = W1.shape[1]
    W3 = _u16(W3, (E, f, h))
    W2 = _u16(W2, (E, h, f))
    F_ref = np.ascontiguousarray(F_ref, dtype=np.float32)
    assert F_ref.shape == (T, h)
    nC = comb(E, r)
    losses = np.zeros(nC, np.float64)
    loss_sq = np.zeros(nC, np.float64)
    best = ctypes.c_uint32(0)
    rc = lib().oracle_prune_search_progressive(
        _p(x_p, _u16p), _p(Wg, _u16p), _p(W1, _u16p), _p(W3, _u16p), _p(W2, _u16p), _p(F_ref, _f32p),
        T, h, f, E, r, _p(losses, _f64p), _p(loss_sq, _f64p), ctypes.byref(best))
    if rc:
        raise ValueError("oracle progressive search: invalid arguments")
    return dict(losses=losses, loss_sq=loss_sq, best_subset=int(best.value), subsets=enumerate_subsets(E, r))


def rmsnorm(x, eps: float = 1e-5) -> np.ndarray:
    x = _u16(x)
    T, h = x.shape
    out = np.zeros((T, h), np.uint16)
    lib().oracle_rmsnorm(_p(x, _u16p), T, h, ctypes.c_double(eps), _p(out, _u16p))
    return out

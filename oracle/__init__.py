"""CPU oracle for per-token routed LoRA -- TEST INFRASTRUCTURE ONLY.

Thin ctypes wrapper over ``molora_oracle.c`` (plain C, fp64, naive per-token loops written from the
paper's definitions).  Only ``tests/``, the smoke check and the benchmark's cpu-baseline / reference
legs may import this package; the CUDA product path never does, and this package imports nothing
from the product package.

Every function takes numpy arrays (float32 values -- exact for bf16-representable data -- and int32
indices) and returns fp64 / int32 numpy arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "molora_oracle.c")
_LIB = os.path.join(_HERE, "libmolora_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math: summation order is part of the definition)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.run(["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"], check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i32p, f32p, f64p, i64p = (ctypes.POINTER(t) for t in (ctypes.c_int32, ctypes.c_float, ctypes.c_double,
                                                                ctypes.c_int64))
        lib.oracle_num_threads.restype = ctypes.c_int
        lib.oracle_route_vocab.argtypes = [i32p, ctypes.c_int64, i32p, ctypes.c_int32, i32p]
        lib.oracle_route_composite.argtypes = [i32p, i32p, ctypes.c_int64, i32p, ctypes.c_int32, ctypes.c_int32, i32p]
        lib.oracle_topk_softmax.argtypes = [f64p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, i32p, f64p]
        lib.oracle_apply_topk.argtypes = [f32p, ctypes.c_int64, f32p, ctypes.c_int64, f32p, f32p, i32p, f64p, ctypes.c_int32,
                                          ctypes.c_int64, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                          ctypes.c_double, f64p]
        lib.oracle_route_mlp.argtypes = [f32p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, f32p, f32p, ctypes.c_int32, f32p,
                                         f32p, ctypes.c_int32, i32p, f64p, f64p, f64p]
        lib.oracle_route_gate.argtypes = [f32p, ctypes.c_int64, ctypes.c_int32, ctypes.c_int64, f32p, f32p,
                                          ctypes.c_int32, i32p, f64p, f64p]
        lib.oracle_group.argtypes = [i32p, ctypes.c_int64, ctypes.c_int32, i32p, i32p, i32p]
        lib.oracle_apply.argtypes = [f32p, ctypes.c_int64, f32p, ctypes.c_int64, f32p, f32p, i32p, ctypes.c_int64,
                                     ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_double,
                                     f64p, i64p]
        lib.oracle_apply_perseq_kpass.argtypes = list(lib.oracle_apply.argtypes)
        _lib = lib
    return _lib


def _p(a: Optional[np.ndarray], ct):
    return None if a is None else a.ctypes.data_as(ctypes.POINTER(ct))


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def route_vocab(ids, breaks) -> np.ndarray:
    """Definition 3.1 (0-based): r[i] = m with breaks[m] <= ids[i] < breaks[m+1]; -1 if no range holds the id."""
    ids, breaks = _i32(ids), _i32(breaks)
    r = np.empty(ids.shape[0], dtype=np.int32)
    rc = _load().oracle_route_vocab(_p(ids, ctypes.c_int32), ids.shape[0], _p(breaks, ctypes.c_int32),
                                    breaks.shape[0] - 1, _p(r, ctypes.c_int32))
    if rc:
        raise ValueError("oracle_route_vocab: invalid arguments")
    return r


def route_composite(ids, adapter, breaks, n_adapters: int) -> np.ndarray:
    """Definition 3.2 / Algorithm 1: r[t] = adapter[t] * M + m(ids[t]); -1 if the id is in no range or the adapter
    index is outside [0, n_adapters)."""
    ids, adapter, breaks = _i32(ids), _i32(adapter), _i32(breaks)
    assert adapter.shape == ids.shape
    r = np.empty(ids.shape[0], dtype=np.int32)
    rc = _load().oracle_route_composite(_p(ids, ctypes.c_int32), _p(adapter, ctypes.c_int32), ids.shape[0],
                                        _p(breaks, ctypes.c_int32), breaks.shape[0] - 1, int(n_adapters),
                                        _p(r, ctypes.c_int32))
    if rc:
        raise ValueError("oracle_route_composite: invalid arguments")
    return r


def route_mlp(x, W1, b1, W2, b2, return_hidden: bool = False):
    """The paper's router (Eq. 9), top-1: g(x) = W2 GELU(W1 x + b1) + b2 with W1 [d, H], W2 [H, C] (input-major) and
    the exact erf GELU.  Returns (r, logits z [N, C] fp64, margin top1 - top2 [N]) (+ hidden [N, H] if asked)."""
    x, W1, W2 = _f32(x), _f32(W1), _f32(W2)
    N, d = x.shape
    H, C = W2.shape
    assert W1.shape == (d, H) and H <= 1024
    b1 = None if b1 is None else _f32(b1)
    b2 = None if b2 is None else _f32(b2)
    r = np.empty(N, dtype=np.int32)
    z = np.empty((N, C), dtype=np.float64)
    margin = np.empty(N, dtype=np.float64)
    h = np.empty((N, H), dtype=np.float64)
    rc = _load().oracle_route_mlp(_p(x, ctypes.c_float), N, d, d, _p(W1, ctypes.c_float), _p(b1, ctypes.c_float), H,
                                  _p(W2, ctypes.c_float), _p(b2, ctypes.c_float), C, _p(r, ctypes.c_int32),
                                  _p(z, ctypes.c_double), _p(margin, ctypes.c_double), _p(h, ctypes.c_double))
    if rc:
        raise ValueError("oracle_route_mlp: invalid arguments")
    return (r, z, margin, h) if return_hidden else (r, z, margin)


def topk_softmax(z, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 8: the k largest logits of every token (ties: lowest index first) and the softmax over them.
    Returns (idx int32 [k, N], w fp64 [k, N]), slot 0 = the largest logit."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    N, C = z.shape
    idx = np.empty((k, N), dtype=np.int32)
    w = np.empty((k, N), dtype=np.float64)
    rc = _load().oracle_topk_softmax(_p(z, ctypes.c_double), N, C, int(k), _p(idx, ctypes.c_int32), _p(w, ctypes.c_double))
    if rc:
        raise ValueError("oracle_topk_softmax: invalid arguments")
    return idx, w


def apply_topk(x, y, A, B, idx, w, scale: float = 1.0) -> np.ndarray:
    """Eq. 8: h_i = y_i + scale * sum_j w[j, i] x_i A[idx[j, i]] B[idx[j, i]] in fp64."""
    x, y, A, B = _f32(x), _f32(y), _f32(A), _f32(B)
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    w = np.ascontiguousarray(w, dtype=np.float64)
    k, N = idx.shape
    C, d_in, rank = A.shape
    d_out = B.shape[2]
    assert x.shape == (N, d_in) and y.shape == (N, d_out) and B.shape == (C, rank, d_out) and w.shape == (k, N)
    h = np.empty((N, d_out), dtype=np.float64)
    rc = _load().oracle_apply_topk(_p(x, ctypes.c_float), d_in, _p(y, ctypes.c_float), d_out, _p(A, ctypes.c_float),
                                   _p(B, ctypes.c_float), _p(idx, ctypes.c_int32), _p(w, ctypes.c_double), k, N, d_in,
                                   d_out, rank, C, float(scale), _p(h, ctypes.c_double))
    if rc:
        raise ValueError("oracle_apply_topk: invalid arguments")
    return h


def route_gate(x, G, bias=None) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Linear gate, top-1 (Eq. 8, k = 1): returns (r, logits z [N, C] fp64, margin top1 - top2 [N])."""
    x, G = _f32(x), _f32(G)
    N, d = x.shape
    C = G.shape[1]
    assert G.shape[0] == d
    b = None if bias is None else _f32(bias)
    r = np.empty(N, dtype=np.int32)
    z = np.empty((N, C), dtype=np.float64)
    margin = np.empty(N, dtype=np.float64)
    rc = _load().oracle_route_gate(_p(x, ctypes.c_float), N, d, d, _p(G, ctypes.c_float), _p(b, ctypes.c_float), C,
                                   _p(r, ctypes.c_int32), _p(z, ctypes.c_double), _p(margin, ctypes.c_double))
    if rc:
        raise ValueError("oracle_route_gate: invalid arguments")
    return r, z, margin


def group(r, C: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Section 3.3: (counts [C], offsets [C+1], perm [#routed]) with ascending token order inside a group."""
    r = _i32(r)
    N = r.shape[0]
    counts = np.empty(C, dtype=np.int32)
    offsets = np.empty(C + 1, dtype=np.int32)
    perm = np.full(max(N, 1), -1, dtype=np.int32)
    rc = _load().oracle_group(_p(r, ctypes.c_int32), N, C, _p(counts, ctypes.c_int32), _p(offsets, ctypes.c_int32),
                              _p(perm, ctypes.c_int32))
    if rc:
        raise ValueError("oracle_group: invalid arguments")
    return counts, offsets, perm[: int(offsets[C])]


def _apply(fn, x, y, A, B, r, scale):
    x, y, A, B, r = _f32(x), _f32(y), _f32(A), _f32(B), _i32(r)
    N, d_in = x.shape
    d_out = y.shape[1]
    C, _, rank = A.shape
    assert A.shape == (C, d_in, rank) and B.shape == (C, rank, d_out) and y.shape[0] == N and r.shape == (N,)
    h = np.empty((N, d_out), dtype=np.float64)
    products = ctypes.c_int64(0)
    rc = fn(_p(x, ctypes.c_float), d_in, _p(y, ctypes.c_float), d_out, _p(A, ctypes.c_float), _p(B, ctypes.c_float),
            _p(r, ctypes.c_int32), N, d_in, d_out, rank, C, float(scale), _p(h, ctypes.c_double),
            ctypes.byref(products))
    if rc:
        raise ValueError("oracle apply: invalid arguments")
    return h, int(products.value)


def apply(x, y, A, B, r, scale: float = 1.0) -> Tuple[np.ndarray, int]:
    """Eq. 2: h_i = y_i + scale * x_i A_{r(i)} B_{r(i)} in fp64, token by token; also the product count."""
    return _apply(_load().oracle_apply, x, y, A, B, r, scale)


def apply_perseq_kpass(x, y, A, B, r, scale: float = 1.0) -> Tuple[np.ndarray, int]:
    """Eq. 1 run once per adapter over all tokens (K passes) with a row mask; also the K*N product count."""
    return _apply(_load().oracle_apply_perseq_kpass, x, y, A, B, r, scale)


def apply_rows(x, y, A, B, r, rows, scale: float = 1.0) -> np.ndarray:
    """Eq. 2 for the selected token rows only (tokens are independent, so a row subset is exact)."""
    rows = np.asarray(rows, dtype=np.int64)
    return apply(np.asarray(x)[rows], np.asarray(y)[rows], A, B, np.asarray(r)[rows], scale)[0]

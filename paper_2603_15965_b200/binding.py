"""ctypes binding of the C ABI in include/molora.h.  Argument marshalling only.

Each ``molora_*`` function mirrors the C entry point of the same name: torch tensors stand for the
device pointers (``data_ptr()``), sizes and pitches are read from their shapes and strides, and the
stream is ``torch.cuda.current_stream()`` unless one is given.  Output tensors are allocated with
torch when the caller does not pass them (device memory is PyTorch's job; the library allocates
nothing).  A non-zero status raises :class:`MoloraError`; a missing shared library raises too --
there is no fallback path.
"""
from __future__ import annotations

import ctypes
import os
import re
from dataclasses import dataclass
from typing import List, Optional, Sequence, Tuple

import torch

from .build import LIB_PATH, ROOT

F32, BF16 = 0, 1
MAX_ADAPTERS = 256
MAX_PROJECTIONS = 8

_lib = None


class MoloraError(RuntimeError):
    def __init__(self, fn: str, status: int, text: str):
        super().__init__(f"{fn} failed: status {status} ({text})")
        self.status = status


class _HostProjC(ctypes.Structure):
    _fields_ = [("x_host", ctypes.c_void_p), ("y_host", ctypes.c_void_p), ("A", ctypes.c_void_p), ("B", ctypes.c_void_p),
                ("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32), ("rank", ctypes.c_int32), ("scale", ctypes.c_float)]


class _ProjDescC(ctypes.Structure):
    _fields_ = [("x", ctypes.c_void_p), ("ldx", ctypes.c_int64), ("y", ctypes.c_void_p), ("ldy", ctypes.c_int64),
                ("A", ctypes.c_void_p), ("B", ctypes.c_void_p), ("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32),
                ("rank", ctypes.c_int32), ("scale", ctypes.c_float), ("row_scale", ctypes.c_void_p)]


COPY_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p)
EVENT_RECORD_FN = ctypes.CFUNCTYPE(ctypes.c_int, ctypes.POINTER(ctypes.c_void_p), ctypes.c_void_p, ctypes.c_void_p)
EVENT_DONE_FN = ctypes.CFUNCTYPE(ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p)
EVENT_DESTROY_FN = ctypes.CFUNCTYPE(None, ctypes.c_void_p, ctypes.c_void_p)


class _HotsetBackendC(ctypes.Structure):
    _fields_ = [("copy_h2d", COPY_FN), ("event_record", EVENT_RECORD_FN), ("event_done", EVENT_DONE_FN),
                ("event_destroy", EVENT_DESTROY_FN), ("user", ctypes.c_void_p)]


def lib_path() -> str:
    return LIB_PATH


def exported_symbols() -> List[str]:
    """Names of the functions include/molora.h declares (parsed from the header)."""
    with open(os.path.join(ROOT, "include", "molora.h")) as f:
        text = f.read()
    names = set(re.findall(r"\b(molora_[a-z_]+)\s*\(", text))
    return sorted(n for n in names if not n.endswith("_t"))          # type names before function-pointer members


def load_library():
    """dlopen the in-tree libmolora.so (built by ``paper_2603_15965_b200.build``) and declare signatures."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2603_15965_b200.build` "
                          "(there is no CPU or PyTorch fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32, sz = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float, ctypes.c_size_t
    lib.molora_version.restype = ctypes.c_char_p
    lib.molora_version.argtypes = []
    lib.molora_status_string.restype = ctypes.c_char_p
    lib.molora_status_string.argtypes = [ctypes.c_int]
    lib.molora_launch_count.restype = ctypes.c_uint64
    lib.molora_launch_count.argtypes = []
    lib.molora_debug_set.restype = ctypes.c_int
    lib.molora_debug_set.argtypes = [ctypes.c_char_p, i64]
    lib.molora_route_vocab.argtypes = [vp, i64, vp, i32, vp, vp, vp]
    lib.molora_route_composite.argtypes = [vp, vp, i64, vp, i32, i32, vp, vp, vp]
    lib.molora_topk_softmax.argtypes = [vp, i64, i32, i32, vp, vp, vp]
    lib.molora_apply_topk_workspace_bytes.restype = sz
    lib.molora_apply_topk_workspace_bytes.argtypes = [vp, i32, i64, i32]
    lib.molora_apply_topk.argtypes = [vp, i32, ctypes.c_int, i64, i32, i32, vp, vp, vp, sz, vp, vp]
    lib.molora_route_mlp_workspace_bytes.restype = sz
    lib.molora_route_mlp_workspace_bytes.argtypes = [ctypes.c_int, i32, i32, i32]
    lib.molora_route_mlp.argtypes = [vp, ctypes.c_int, i64, i32, i64, vp, vp, i32, vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.molora_route_gate_workspace_bytes.restype = sz
    lib.molora_route_gate_workspace_bytes.argtypes = [ctypes.c_int, i32, i32]
    lib.molora_route_gate.argtypes = [vp, ctypes.c_int, i64, i32, i64, vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.molora_route_gate_prepared_workspace_bytes.restype = sz
    lib.molora_route_gate_prepared_workspace_bytes.argtypes = [ctypes.c_int, i32, i32]
    lib.molora_route_gate_prepare.argtypes = [ctypes.c_int, i32, i32, vp, vp, sz, vp]
    lib.molora_route_gate_prepared.argtypes = [vp, ctypes.c_int, i64, i32, i64, vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.molora_route_mlp_prepare.argtypes = [ctypes.c_int, i32, i32, i32, vp, vp, sz, vp]
    lib.molora_route_mlp_prepared.argtypes = [vp, ctypes.c_int, i64, i32, i64, vp, vp, i32, vp, vp, i32, vp, vp, vp, sz, vp, vp]
    lib.molora_route_gate_noalloc.argtypes = [vp, ctypes.c_int, i64, i32, i64, vp, vp, i32, vp, vp, vp]
    lib.molora_route_gate_noalloc.restype = ctypes.c_int
    lib.molora_selftest_bounded_wait.argtypes = [vp, i64, vp, vp]
    lib.molora_selftest_bounded_wait.restype = ctypes.c_int
    lib.molora_group_workspace_bytes.restype = sz
    lib.molora_group_workspace_bytes.argtypes = [i64, i32]
    lib.molora_group.argtypes = [vp, i64, i32, vp, vp, vp, vp, sz, vp, vp]
    lib.molora_apply_workspace_bytes.restype = sz
    lib.molora_apply_workspace_bytes.argtypes = [i64, i32, i32, i32, i32]
    lib.molora_apply.argtypes = [vp, i64, vp, i64, ctypes.c_int, i64, i32, i32, i32, vp, vp, i32, vp, vp, f32, vp, sz,
                                 vp, vp]
    lib.molora_apply_batched.argtypes = [ctypes.POINTER(_ProjDescC), i32, ctypes.c_int, i64, i32, vp, vp, vp, sz, vp,
                                         vp]
    lib.molora_group_apply_batched.argtypes = [vp, i64, i32, vp, vp, vp, ctypes.POINTER(_ProjDescC), i32, ctypes.c_int, vp,
                                               sz, vp, vp]
    lib.molora_group_apply_batched.restype = ctypes.c_int
    lib.molora_group_apply_is_one_launch.argtypes = [ctypes.POINTER(_ProjDescC), i32, ctypes.c_int, i64, i32]
    lib.molora_group_apply_is_one_launch.restype = i32
    lib.molora_group_apply_skips_group_launch.argtypes = [ctypes.POINTER(_ProjDescC), i32, ctypes.c_int, i64, i32]
    lib.molora_group_apply_skips_group_launch.restype = i32
    lib.molora_forward_host_arena_bytes.restype = sz
    lib.molora_forward_host_arena_bytes.argtypes = [ctypes.POINTER(_HostProjC), i32, ctypes.c_int, i64, i32, ctypes.c_int,
                                                    i32]
    lib.molora_forward_host.argtypes = [ctypes.c_int, vp, vp, i32, vp, vp, i32, ctypes.POINTER(_HostProjC), i32,
                                        ctypes.c_int, i64, i32, vp, sz, vp, vp]
    lib.molora_hotset_create.argtypes = [i32, i32, i32, vp, ctypes.POINTER(_HotsetBackendC), ctypes.POINTER(vp)]
    lib.molora_hotset_destroy.argtypes = [vp]
    lib.molora_hotset_destroy.restype = None
    lib.molora_hotset_slot_of.argtypes = [vp, i32]
    lib.molora_hotset_slot_of.restype = i32
    lib.molora_hotset_adapter_in.argtypes = [vp, i32]
    lib.molora_hotset_adapter_in.restype = i32
    lib.molora_hotset_pin.argtypes = [vp, i32, ctypes.POINTER(i32)]
    lib.molora_hotset_unpin.argtypes = [vp, i32]
    lib.molora_hotset_begin_load.argtypes = [vp, i32, vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i32)]
    lib.molora_hotset_upload.argtypes = [vp, i32, vp, vp, sz, vp]
    lib.molora_hotset_commit.argtypes = [vp, i32, vp]
    lib.molora_route_hotset.argtypes = [vp, vp, i64, vp, i32, vp, i32, i32, vp, vp, vp]
    for name in ("molora_hotset_create", "molora_hotset_pin", "molora_hotset_unpin", "molora_hotset_begin_load",
                 "molora_hotset_upload", "molora_hotset_commit", "molora_route_hotset"):
        getattr(lib, name).restype = ctypes.c_int
    for name in ("molora_route_vocab", "molora_route_gate", "molora_group", "molora_apply", "molora_apply_batched",
                 "molora_forward_host"):
        getattr(lib, name).restype = ctypes.c_int
    _lib = lib
    return lib


# ----------------------------------------------------------------------------- helpers
def _check(fn: str, status: int) -> None:
    if status != 0:
        raise MoloraError(fn, status, load_library().molora_status_string(status).decode())


def _stream(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported element type {t.dtype}: fp32 or bf16 only")


def _matrix(t: torch.Tensor, name: str) -> Tuple[int, int, int]:
    """(rows, cols, pitch in elements) of a 2-D row-major device tensor."""
    if not t.is_cuda or t.dim() != 2 or (t.shape[1] > 1 and t.stride(1) != 1):
        raise ValueError(f"{name}: expected a 2-D row-major CUDA tensor")
    return t.shape[0], t.shape[1], (t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1]))


def _i32_dev(t: torch.Tensor, name: str) -> torch.Tensor:
    if not t.is_cuda or t.dtype != torch.int32 or not t.is_contiguous():
        raise ValueError(f"{name}: expected a contiguous int32 CUDA tensor")
    return t


# ----------------------------------------------------------------------------- entry points
def molora_version() -> str:
    return load_library().molora_version().decode()


def molora_launch_count() -> int:
    """Kernels the library has enqueued in this process so far."""
    return int(load_library().molora_launch_count())


TUNING_NAMES = ("umma_min_tokens", "small_path", "stream_tile", "umma_split", "umma_tile_rows", "group_split",
                "chained_launch_off", "jobs_launch")


def molora_debug_set(name: str, value: int) -> None:
    """Override one of the library's kernel choices (0 = default); see include/molora.h."""
    _check("molora_debug_set", load_library().molora_debug_set(name.encode(), int(value)))


def molora_status_string(status: int) -> str:
    return load_library().molora_status_string(int(status)).decode()


def molora_route_vocab(ids: torch.Tensor, breaks: torch.Tensor, r_out: Optional[torch.Tensor] = None,
                       dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """r_out[i] = m with breaks[m] <= ids[i] < breaks[m+1] (Definition 3.1, 0-based); -1 if unrouted."""
    lib = load_library()
    _i32_dev(ids, "ids"), _i32_dev(breaks, "breaks")
    N, M = ids.numel(), breaks.numel() - 1
    if r_out is None:
        r_out = torch.empty(N, dtype=torch.int32, device=ids.device)
    _check("molora_route_vocab", lib.molora_route_vocab(_ptr(ids), N, _ptr(breaks), M, _ptr(_i32_dev(r_out, "r_out")),
                                                        _ptr(dev_status), _stream(stream)))
    return r_out


def molora_route_composite(ids: torch.Tensor, adapter: torch.Tensor, breaks: torch.Tensor, n_adapters: int,
                           r_out: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                           stream=None) -> torch.Tensor:
    """r_out[i] = adapter[i] * M + m(ids[i]) (Definition 3.2 / Algorithm 1); -1 if the token is unrouted."""
    lib = load_library()
    _i32_dev(ids, "ids"), _i32_dev(adapter, "adapter"), _i32_dev(breaks, "breaks")
    N, M = ids.numel(), breaks.numel() - 1
    if adapter.numel() != N:
        raise ValueError("adapter must hold one index per token")
    if r_out is None:
        r_out = torch.empty(N, dtype=torch.int32, device=ids.device)
    _check("molora_route_composite", lib.molora_route_composite(_ptr(ids), _ptr(adapter), N, _ptr(breaks), M,
                                                                int(n_adapters), _ptr(_i32_dev(r_out, "r_out")),
                                                                _ptr(dev_status), _stream(stream)))
    return r_out


def molora_route_mlp_workspace_bytes(xdt: int, d: int, H: int, C: int) -> int:
    return int(load_library().molora_route_mlp_workspace_bytes(xdt, d, H, C))


def molora_route_mlp(x: torch.Tensor, W1: torch.Tensor, b1: Optional[torch.Tensor], W2: torch.Tensor,
                     b2: Optional[torch.Tensor], r_out: Optional[torch.Tensor] = None,
                     logits_out: Optional[torch.Tensor] = None, ws: Optional[torch.Tensor] = None,
                     dev_status: Optional[torch.Tensor] = None, stream=None, prepared: Optional[torch.Tensor] = None) -> torch.Tensor:
    """r_out[i] = argmax_c (W2 GELU(W1 x_i + b1) + b2)[c] (Eq. 9, top-1); W1 [d, H], W2 [H, C] fp32.
    ``prepared``: the workspace molora_route_mlp_prepare returned for this W1 (saves the preparation launch)."""
    lib = load_library()
    N, d, ldx = _matrix(x, "x")
    if W1.dtype != torch.float32 or W2.dtype != torch.float32 or not W1.is_contiguous() or not W2.is_contiguous():
        raise ValueError("W1 [d, H] and W2 [H, C] must be dense fp32 tensors")
    H, C = W2.shape
    if tuple(W1.shape) != (d, H):
        raise ValueError("W1 must be [d, H]")
    if r_out is None:
        r_out = torch.empty(N, dtype=torch.int32, device=x.device)
    need = molora_route_mlp_workspace_bytes(_dtype_code(x), d, H, C)
    if ws is None and need > 0:
        ws = torch.zeros(need, dtype=torch.uint8, device=x.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    if prepared is not None:
        _check("molora_route_mlp_prepared", lib.molora_route_mlp_prepared(
            _ptr(x), _dtype_code(x), N, d, ldx, _ptr(W1), _ptr(b1), H, _ptr(W2), _ptr(b2), C, _ptr(_i32_dev(r_out, "r_out")),
            _ptr(logits_out), _ptr(prepared), prepared.numel(), _ptr(dev_status), _stream(stream)))
        return r_out
    _check("molora_route_mlp", lib.molora_route_mlp(_ptr(x), _dtype_code(x), N, d, ldx, _ptr(W1), _ptr(b1), H, _ptr(W2),
                                                    _ptr(b2), C, _ptr(_i32_dev(r_out, "r_out")), _ptr(logits_out),
                                                    _ptr(ws), ws_bytes, _ptr(dev_status), _stream(stream)))
    return r_out


def molora_route_gate_workspace_bytes(xdt: int, d: int, C: int) -> int:
    return int(load_library().molora_route_gate_workspace_bytes(xdt, d, C))


def molora_route_gate(x: torch.Tensor, G: torch.Tensor, bias: Optional[torch.Tensor] = None,
                      r_out: Optional[torch.Tensor] = None, logits_out: Optional[torch.Tensor] = None,
                      ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                      stream=None, prepared: Optional[torch.Tensor] = None) -> torch.Tensor:
    """r_out[i] = argmax_c sum_k x[i,k] G[k,c] (+ bias[c]) (Eq. 8, k = 1); lowest index on ties.
    ``prepared``: the workspace molora_route_gate_prepare returned for this G (saves the preparation launch)."""
    lib = load_library()
    N, d, ldx = _matrix(x, "x")
    if G.dtype != torch.float32 or not G.is_cuda or not G.is_contiguous() or G.dim() != 2 or G.shape[0] != d:
        raise ValueError("G: expected a contiguous fp32 CUDA tensor of shape [d, C]")
    C = G.shape[1]
    if bias is not None and (bias.dtype != torch.float32 or bias.numel() != C or not bias.is_contiguous()):
        raise ValueError("bias: expected contiguous fp32 [C]")
    if r_out is None:
        r_out = torch.empty(N, dtype=torch.int32, device=x.device)
    if logits_out is not None and (logits_out.dtype != torch.float32 or logits_out.shape != (N, C)
                                   or not logits_out.is_contiguous()):
        raise ValueError("logits_out: expected contiguous fp32 [N, C]")
    if prepared is not None:
        _check("molora_route_gate_prepared", lib.molora_route_gate_prepared(
            _ptr(x), _dtype_code(x), N, d, ldx, _ptr(G), _ptr(bias), C, _ptr(_i32_dev(r_out, "r_out")), _ptr(logits_out),
            _ptr(prepared), prepared.numel(), _ptr(dev_status), _stream(stream)))
        return r_out
    need = molora_route_gate_workspace_bytes(_dtype_code(x), d, C)
    if ws is None and need > 0:
        ws = torch.zeros(need, dtype=torch.uint8, device=x.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check("molora_route_gate", lib.molora_route_gate(_ptr(x), _dtype_code(x), N, d, ldx, _ptr(G), _ptr(bias), C,
                                                      _ptr(_i32_dev(r_out, "r_out")), _ptr(logits_out), _ptr(ws),
                                                      ws_bytes, _ptr(dev_status), _stream(stream)))
    return r_out


def molora_route_gate_prepare(x_dtype: torch.dtype, G: torch.Tensor, ws: Optional[torch.Tensor] = None, stream=None):
    """Build the gate's weight images once (static router weights); returns the workspace to pass to
    molora_route_gate(..., prepared=ws).  None when this gate needs no image (fp32 activations or at most 4 adapters)."""
    lib = load_library()
    if G.dtype != torch.float32 or not G.is_cuda or not G.is_contiguous() or G.dim() != 2:
        raise ValueError("G: expected a contiguous fp32 CUDA tensor of shape [d, C]")
    d, C = G.shape
    xdt = BF16 if x_dtype == torch.bfloat16 else F32
    need = int(lib.molora_route_gate_prepared_workspace_bytes(xdt, d, C))
    if need == 0:
        return None
    if ws is None:
        ws = torch.empty(need, dtype=torch.uint8, device=G.device)
    _check("molora_route_gate_prepare", lib.molora_route_gate_prepare(xdt, d, C, _ptr(G), _ptr(ws), ws.numel(), _stream(stream)))
    return ws


def molora_route_mlp_prepare(x_dtype: torch.dtype, W1: torch.Tensor, C: int, ws: Optional[torch.Tensor] = None, stream=None):
    """Build the MLP router's first-layer images once; returns the workspace for molora_route_mlp(..., prepared=ws)."""
    lib = load_library()
    if W1.dtype != torch.float32 or not W1.is_cuda or not W1.is_contiguous() or W1.dim() != 2:
        raise ValueError("W1: expected a contiguous fp32 CUDA tensor of shape [d, H]")
    d, H = W1.shape
    xdt = BF16 if x_dtype == torch.bfloat16 else F32
    need = molora_route_mlp_workspace_bytes(xdt, d, H, C)
    if need == 0:
        return None
    if ws is None:
        ws = torch.empty(need, dtype=torch.uint8, device=W1.device)
    _check("molora_route_mlp_prepare", lib.molora_route_mlp_prepare(xdt, d, H, C, _ptr(W1), _ptr(ws), ws.numel(), _stream(stream)))
    return ws


def molora_route_gate_noalloc(x: torch.Tensor, G: torch.Tensor, bias: Optional[torch.Tensor] = None,
                              r_out: Optional[torch.Tensor] = None, logits_out: Optional[torch.Tensor] = None,
                              stream=None) -> torch.Tensor:
    """The gate without a caller workspace: its scratch is a fixed 2 MiB array inside the library (so gates whose
    split weights need more are refused), for callers that cannot allocate device memory where they route.
    Pass ``r_out`` to keep this binding allocation-free as well.  Calls that overlap on the GPU race on the array."""
    lib = load_library()
    N, d, ldx = _matrix(x, "x")
    if G.dtype != torch.float32 or not G.is_cuda or not G.is_contiguous() or G.dim() != 2 or G.shape[0] != d:
        raise ValueError("G: expected a contiguous fp32 CUDA tensor of shape [d, C]")
    C = G.shape[1]
    if r_out is None:
        r_out = torch.empty(N, dtype=torch.int32, device=x.device)
    _check("molora_route_gate_noalloc", lib.molora_route_gate_noalloc(
        _ptr(x), _dtype_code(x), N, d, ldx, _ptr(G), _ptr(bias), C, _ptr(_i32_dev(r_out, "r_out")), _ptr(logits_out),
        _stream(stream)))
    return r_out


def molora_selftest_bounded_wait(limit_cycles: int = 200000, stream=None) -> Tuple[int, int, int]:
    """Run the bounded-wait self-test; returns (status word, abort flag, second wait fell through)."""
    lib = load_library()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    result = torch.zeros(2, dtype=torch.int32, device="cuda")
    _check("molora_selftest_bounded_wait", lib.molora_selftest_bounded_wait(_ptr(status), int(limit_cycles), _ptr(result),
                                                                            _stream(stream)))
    torch.cuda.synchronize()
    return int(status.item()), int(result[0].item()), int(result[1].item())


def molora_group_workspace_bytes(N: int, C: int) -> int:
    return int(load_library().molora_group_workspace_bytes(N, C))


def molora_group(r: torch.Tensor, C: int, counts: Optional[torch.Tensor] = None,
                 offsets: Optional[torch.Tensor] = None, perm: Optional[torch.Tensor] = None,
                 ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None,
                 stream=None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """(counts [C], offsets [C+1], perm [N]) of Section 3.3; perm is stable, its first offsets[C] entries valid."""
    lib = load_library()
    _i32_dev(r, "r")
    N = r.numel()
    dev = r.device
    counts = torch.empty(C, dtype=torch.int32, device=dev) if counts is None else _i32_dev(counts, "counts")
    offsets = torch.empty(C + 1, dtype=torch.int32, device=dev) if offsets is None else _i32_dev(offsets, "offsets")
    perm = torch.empty(max(N, 1), dtype=torch.int32, device=dev) if perm is None else _i32_dev(perm, "perm")
    need = molora_group_workspace_bytes(N, C)
    if ws is None and need > 0:
        ws = torch.zeros(need, dtype=torch.uint8, device=dev)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check("molora_group", lib.molora_group(_ptr(r), N, C, _ptr(counts), _ptr(offsets), _ptr(perm), _ptr(ws), ws_bytes,
                                            _ptr(dev_status), _stream(stream)))
    return counts, offsets, perm


def molora_apply_workspace_bytes(N: int, C: int, d_in: int, d_out: int, rank: int) -> int:
    return int(load_library().molora_apply_workspace_bytes(N, C, d_in, d_out, rank))


def molora_apply(x: torch.Tensor, y: torch.Tensor, A: torch.Tensor, B: torch.Tensor, offsets: torch.Tensor,
                 perm: torch.Tensor, scale: float = 1.0, ws: Optional[torch.Tensor] = None,
                 dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """In place: y[i] += scale * (x[i] A[c]) B[c] for every token i of every segment c (Eq. 2).  Returns y."""
    lib = load_library()
    N, d_in, ldx = _matrix(x, "x")
    Ny, d_out, ldy = _matrix(y, "y")
    dt = _dtype_code(x)
    if Ny != N or y.dtype != x.dtype or A.dtype != x.dtype or B.dtype != x.dtype:
        raise ValueError("x, y, A, B must share the token count and the element type")
    if A.dim() != 3 or B.dim() != 3 or not A.is_contiguous() or not B.is_contiguous():
        raise ValueError("A [C, d_in, rank] and B [C, rank, d_out] must be dense 3-D tensors")
    C, rank = A.shape[0], A.shape[2]
    if A.shape[1] != d_in or tuple(B.shape) != (C, rank, d_out):
        raise ValueError("A / B shapes do not match x / y")
    if offsets.numel() != C + 1:
        raise ValueError("offsets must have C + 1 entries")
    need = molora_apply_workspace_bytes(N, C, d_in, d_out, rank)
    if ws is None and need > 0:
        ws = torch.zeros(need, dtype=torch.uint8, device=x.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check("molora_apply", lib.molora_apply(_ptr(x), ldx, _ptr(y), ldy, dt, N, d_in, d_out, rank, _ptr(A), _ptr(B), C,
                                            _ptr(_i32_dev(offsets, "offsets")), _ptr(_i32_dev(perm, "perm")),
                                            float(scale), _ptr(ws), ws_bytes, _ptr(dev_status), _stream(stream)))
    return y


@dataclass
class ProjDesc:
    """One projection of a batched apply: tensors as in :func:`molora_apply`."""
    x: torch.Tensor
    y: torch.Tensor
    A: torch.Tensor
    B: torch.Tensor
    scale: float = 1.0
    row_scale: Optional[torch.Tensor] = None     # fp32 [N]: extra per-token factor on the delta (top-k routing weights)


def pack_proj_descs(projs: Sequence[ProjDesc]):
    """Marshal ProjDesc objects into the C descriptor array (reusable across calls while the tensors live)."""
    arr = (_ProjDescC * len(projs))()
    N = C = dt = None
    for i, p in enumerate(projs):
        n, d_in, ldx = _matrix(p.x, "x")
        ny, d_out, ldy = _matrix(p.y, "y")
        if ny != n or p.y.dtype != p.x.dtype or p.A.dtype != p.x.dtype or p.B.dtype != p.x.dtype:
            raise ValueError("x, y, A, B must share the token count and the element type")
        c, rank = p.A.shape[0], p.A.shape[2]
        if (not p.A.is_contiguous() or not p.B.is_contiguous() or p.A.shape[1] != d_in
                or tuple(p.B.shape) != (c, rank, d_out)):
            raise ValueError("A / B shapes do not match x / y")
        if N is None:
            N, C, dt = n, c, _dtype_code(p.x)
        elif (N, C, dt) != (n, c, _dtype_code(p.x)):
            raise ValueError("all projections of a batched apply share N, C and the element type")
        rs = getattr(p, "row_scale", None)
        if rs is not None and (rs.dtype != torch.float32 or rs.numel() != n or not rs.is_contiguous()):
            raise ValueError("row_scale must be a dense fp32 tensor with one factor per token")
        arr[i] = _ProjDescC(p.x.data_ptr(), ldx, p.y.data_ptr(), ldy, p.A.data_ptr(), p.B.data_ptr(), d_in, d_out,
                            rank, float(p.scale), rs.data_ptr() if rs is not None else None)
    return arr, N, C, dt


def molora_apply_batched_workspace_bytes(arr, N: int, C: int) -> int:
    """Scratch a batched apply needs: the sum of molora_apply_workspace_bytes over its projections."""
    return sum(molora_apply_workspace_bytes(N, C, d.d_in, d.d_out, d.rank) for d in arr)


def molora_apply_batched(projs, offsets: torch.Tensor, perm: torch.Tensor, ws: Optional[torch.Tensor] = None,
                         dev_status: Optional[torch.Tensor] = None, stream=None, packed=None) -> None:
    """One launch for the projections of a layer (shared N, C, offsets, perm).  ``projs``: ProjDesc list."""
    lib = load_library()
    arr, N, C, dt = packed if packed is not None else pack_proj_descs(projs)
    if ws is None:
        need = molora_apply_batched_workspace_bytes(arr, N, C)
        if need > 0:
            ws = torch.zeros(need, dtype=torch.uint8, device=offsets.device)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check("molora_apply_batched", lib.molora_apply_batched(arr, len(arr), dt, N, C, _ptr(offsets), _ptr(perm),
                                                            _ptr(ws), ws_bytes, _ptr(dev_status), _stream(stream)))


def molora_group_apply_batched(r: torch.Tensor, projs, C: Optional[int] = None, counts: Optional[torch.Tensor] = None,
                               offsets: Optional[torch.Tensor] = None, perm: Optional[torch.Tensor] = None,
                               ws: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None, stream=None,
                               packed=None) -> Tuple[torch.Tensor, torch.Tensor, torch.Tensor]:
    """molora_group followed by molora_apply_batched as one call (one launch where the library can fuse them).
    Returns (counts, offsets, perm) as molora_group does."""
    lib = load_library()
    _i32_dev(r, "r")
    arr, N, C_, dt = packed if packed is not None else pack_proj_descs(projs)
    C = C_ if C is None else C
    if r.numel() != N or C != C_:
        raise ValueError("r must hold one routing decision per token of the projections")
    dev = r.device
    counts = torch.empty(C, dtype=torch.int32, device=dev) if counts is None else _i32_dev(counts, "counts")
    offsets = torch.empty(C + 1, dtype=torch.int32, device=dev) if offsets is None else _i32_dev(offsets, "offsets")
    perm = torch.empty(max(N, 1), dtype=torch.int32, device=dev) if perm is None else _i32_dev(perm, "perm")
    if ws is None:
        need = molora_apply_batched_workspace_bytes(arr, N, C)
        if need > 0:
            ws = torch.zeros(need, dtype=torch.uint8, device=dev)
    ws_bytes = 0 if ws is None else ws.numel() * ws.element_size()
    _check("molora_group_apply_batched",
           lib.molora_group_apply_batched(_ptr(r), N, C, _ptr(counts), _ptr(offsets), _ptr(perm), arr, len(arr), dt, _ptr(ws),
                                          ws_bytes, _ptr(dev_status), _stream(stream)))
    return counts, offsets, perm


def molora_topk_softmax(logits: torch.Tensor, k: int, stream=None):
    """Eq. 8: the k largest logits per token (ties: lowest index first) and the softmax over them.
    Returns (idx int32 [k, N], w fp32 [k, N]), slot 0 = the largest logit."""
    lib = load_library()
    if logits.dtype != torch.float32 or logits.dim() != 2 or not logits.is_contiguous():
        raise ValueError("logits must be a dense fp32 [N, C] tensor")
    N, C = logits.shape
    idx = torch.empty(k, N, dtype=torch.int32, device=logits.device)
    w = torch.empty(k, N, dtype=torch.float32, device=logits.device)
    _check("molora_topk_softmax", lib.molora_topk_softmax(_ptr(logits), N, C, int(k), _ptr(idx), _ptr(w), _stream(stream)))
    return idx, w


def molora_apply_topk(projs, idx: torch.Tensor, w: torch.Tensor, C: int, ws: Optional[torch.Tensor] = None,
                      dev_status: Optional[torch.Tensor] = None, stream=None) -> None:
    """Eq. 8: y_i += sum_j w[j, i] * scale * (x_i A[idx[j, i]]) B[idx[j, i]] as k passes of (group, apply)."""
    lib = load_library()
    arr, N, C_, dt = pack_proj_descs(projs)
    if C_ != C or idx.dtype != torch.int32 or w.dtype != torch.float32 or tuple(idx.shape) != tuple(w.shape) or idx.shape[1] != N:
        raise ValueError("idx int32 [k, N] and w fp32 [k, N] must match the projections")
    k = idx.shape[0]
    need = int(lib.molora_apply_topk_workspace_bytes(arr, len(arr), N, C))
    if ws is None:
        ws = torch.zeros(need + 256, dtype=torch.uint8, device=idx.device)
    off = (-ws.data_ptr()) % 256
    _check("molora_apply_topk", lib.molora_apply_topk(arr, len(arr), dt, N, C, k, _ptr(idx.contiguous()), _ptr(w.contiguous()),
                                                      ctypes.c_void_p(ws.data_ptr() + off), ws.numel() - off,
                                                      _ptr(dev_status), _stream(stream)))


ROUTE_VOCAB, ROUTE_GATE, ROUTE_GIVEN = 0, 1, 2


@dataclass
class HostProj:
    """One projection of :func:`molora_forward_host`: x, y dense HOST tensors (pinned for asynchronous copies),
    A, B dense DEVICE tensors."""
    x: torch.Tensor
    y: torch.Tensor
    A: torch.Tensor
    B: torch.Tensor
    scale: float = 1.0


def pack_host_projs(projs: Sequence[HostProj]):
    arr = (_HostProjC * len(projs))()
    N = C = dt = None
    for i, p in enumerate(projs):
        if p.x.is_cuda or p.y.is_cuda or not p.x.is_contiguous() or not p.y.is_contiguous():
            raise ValueError("x, y: expected dense host tensors")
        if not p.A.is_cuda or not p.B.is_cuda or not p.A.is_contiguous() or not p.B.is_contiguous():
            raise ValueError("A, B: expected dense device tensors")
        n, d_in = p.x.shape
        d_out = p.y.shape[1]
        c, rank = p.A.shape[0], p.A.shape[2]
        if p.y.shape[0] != n or p.A.shape[1] != d_in or tuple(p.B.shape) != (c, rank, d_out):
            raise ValueError("shapes of x, y, A, B do not match")
        if N is None:
            N, C, dt = n, c, _dtype_code(p.x)
        elif (N, C, dt) != (n, c, _dtype_code(p.x)):
            raise ValueError("all projections share N, C and the element type")
        arr[i] = _HostProjC(p.x.data_ptr(), p.y.data_ptr(), p.A.data_ptr(), p.B.data_ptr(), d_in, d_out, rank,
                            float(p.scale))
    return arr, N, C, dt


def molora_forward_host_arena_bytes(projs, router: int, gate_proj: int = 0, packed=None) -> int:
    arr, N, C, dt = packed if packed is not None else pack_host_projs(projs)
    return int(load_library().molora_forward_host_arena_bytes(arr, len(arr), dt, N, C, router, gate_proj))


def molora_forward_host(router: int, projs, arena: torch.Tensor, route_src: Optional[torch.Tensor] = None,
                        breaks: Optional[torch.Tensor] = None, G: Optional[torch.Tensor] = None,
                        bias: Optional[torch.Tensor] = None, gate_proj: int = 0,
                        dev_status: Optional[torch.Tensor] = None, stream=None, packed=None) -> None:
    """route -> group -> apply on HOST activations (copied in and out on the stream).  Asynchronous."""
    lib = load_library()
    arr, N, C, dt = packed if packed is not None else pack_host_projs(projs)
    M = 0 if breaks is None else breaks.numel() - 1
    _check("molora_forward_host", lib.molora_forward_host(
        router, _ptr(route_src), _ptr(breaks), M, _ptr(G), _ptr(bias), gate_proj, arr, len(arr), dt, N, C,
        _ptr(arena), arena.numel() * arena.element_size(), _ptr(dev_status), _stream(stream)))


# ----------------------------------------------------------------------------- hot-set slot table (Definition 5.1)
ERR_BUSY, ERR_NOT_RESIDENT = 5, 6


class HotSet:
    """Handle of a molora_hotset_t: S slots x M modalities over a catalog of n_catalog adapters.  ``table`` is the device
    int32[n_catalog] inverse slot table (filled with -1 by the caller); with ``backend`` (a _HotsetBackendC of callbacks)
    the copies and events go there instead of the CUDA runtime.  Marshalling only: every decision is the library's."""

    def __init__(self, S: int, M: int, n_catalog: int, table, backend=None):
        self.lib = load_library()
        self.S, self.M, self.n_catalog, self.table, self._backend = S, M, n_catalog, table, backend
        h = ctypes.c_void_p()
        tptr = table.data_ptr() if hasattr(table, "data_ptr") else int(table)
        _check("molora_hotset_create", self.lib.molora_hotset_create(S, M, n_catalog, ctypes.c_void_p(tptr),
                                                                      ctypes.byref(backend) if backend is not None else None,
                                                                      ctypes.byref(h)))
        self.h = h

    def close(self):
        if self.h:
            self.lib.molora_hotset_destroy(self.h)
            self.h = None

    def __del__(self):
        self.close()

    def slot_of(self, adapter: int) -> int:
        return int(self.lib.molora_hotset_slot_of(self.h, adapter))

    def adapter_in(self, slot: int) -> int:
        return int(self.lib.molora_hotset_adapter_in(self.h, slot))

    def pin(self, adapter: int) -> int:
        slot = ctypes.c_int32(-1)
        _check("molora_hotset_pin", self.lib.molora_hotset_pin(self.h, adapter, ctypes.byref(slot)))
        return slot.value

    def unpin(self, slot: int) -> None:
        _check("molora_hotset_unpin", self.lib.molora_hotset_unpin(self.h, slot))

    def begin_load(self, adapter: int, stream=None) -> Tuple[int, bool, int]:
        """Returns (slot, fresh, evicted adapter or -1): upload and commit only when fresh; raises MoloraError with status
        ERR_BUSY if no slot can be had."""
        slot, fresh, ev = ctypes.c_int32(-1), ctypes.c_int32(0), ctypes.c_int32(-1)
        _check("molora_hotset_begin_load", self.lib.molora_hotset_begin_load(self.h, adapter, ctypes.c_void_p(_stream_or_raw(stream)),
                                                                              ctypes.byref(slot), ctypes.byref(fresh), ctypes.byref(ev)))
        return slot.value, bool(fresh.value), ev.value

    def upload(self, slot: int, stack, weights_host, stream=None) -> None:
        """Copy one adapter's weights (host tensor shaped like stack[slot]) into stack[slot] on the maintenance stream."""
        nbytes = weights_host.numel() * weights_host.element_size()
        if hasattr(stack, "shape") and nbytes != stack[0].numel() * stack.element_size():
            raise ValueError("weights do not have the size of one slot of the stack")
        _check("molora_hotset_upload", self.lib.molora_hotset_upload(self.h, slot, ctypes.c_void_p(stack.data_ptr()),
                                                                      ctypes.c_void_p(weights_host.data_ptr()), nbytes,
                                                                      ctypes.c_void_p(_stream_or_raw(stream))))

    def commit(self, slot: int, stream=None) -> None:
        _check("molora_hotset_commit", self.lib.molora_hotset_commit(self.h, slot, ctypes.c_void_p(_stream_or_raw(stream))))


def _stream_or_raw(stream) -> int:
    if stream is None:
        return torch.cuda.current_stream().cuda_stream if torch.cuda.is_available() else 0
    return stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream)


def molora_route_hotset(ids: torch.Tensor, adapter_id: torch.Tensor, breaks: torch.Tensor, slot_table: torch.Tensor, S: int,
                        r_out: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """r[i] = slot_table[adapter_id[i]] * M + modality(ids[i]); -1 where the adapter is not resident."""
    lib = load_library()
    N, M = ids.numel(), breaks.numel() - 1
    if r_out is None:
        r_out = torch.empty(N, dtype=torch.int32, device=ids.device)
    _check("molora_route_hotset", lib.molora_route_hotset(_ptr(_i32_dev(ids, "ids")), _ptr(_i32_dev(adapter_id, "adapter_id")), N,
                                                          _ptr(_i32_dev(breaks, "breaks")), M, _ptr(_i32_dev(slot_table, "slot_table")),
                                                          slot_table.numel(), S, _ptr(r_out), _ptr(dev_status), _stream(stream)))
    return r_out

"""Shared helpers of the GPU parity tests: upload a workload, run the CUDA path through the C ABI
binding, and compare with the CPU oracle.  (The CUDA path never sees the oracle; only the tests do.)"""
from __future__ import annotations

import numpy as np
import torch

import oracle
import paper_2603_15965_b200 as M
from paper_2603_15965_b200 import workloads as W

ATOL, RTOL = 1e-3, 2e-2            # |gpu - ref| <= ATOL + RTOL * |ref|  (bf16 in / fp32 accumulate)
ATOL32, RTOL32 = 1e-5, 1e-4        # tighter bound also required of fp32 storage
GATE_MARGIN = 1e-3                 # learned-gate tokens with a smaller oracle top-2 margin are counted and excluded


def dev_tensor(a: np.ndarray, dtype: str) -> torch.Tensor:
    if a.dtype == np.int32:
        return torch.from_numpy(np.ascontiguousarray(a)).cuda()
    if dtype == "bf16":
        return torch.from_numpy(W.bf16_bits(a)).cuda().view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()


def to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy().astype(np.float64)


def gpu_route(w: W.Workload, status=None):
    """Run the workload's router on the GPU; returns r (device int32)."""
    if w.router == "vocab":
        return M.molora_route_vocab(dev_tensor(w.ids, "i"), dev_tensor(w.breaks, "i"), dev_status=status)
    if w.router == "gate":
        return M.molora_route_gate(dev_tensor(w.inputs[w.gate_x_key], w.dtype), dev_tensor(w.G, "f32"))
    return dev_tensor(w.r, "i")


def oracle_route(w: W.Workload):
    """(r, margin or None) from the oracle."""
    if w.router == "vocab":
        return oracle.route_vocab(w.ids, w.breaks), None
    if w.router == "gate":
        r, _, margin = oracle.route_gate(w.inputs[w.gate_x_key], w.G)
        return r, margin
    return w.r.copy(), None


def assert_close(gpu: np.ndarray, ref: np.ndarray, atol=ATOL, rtol=RTOL, what=""):
    err = np.abs(gpu - ref)
    bound = atol + rtol * np.abs(ref)
    bad = err > bound
    if bad.any():
        i = np.unravel_index(np.argmax(err - bound), err.shape)
        raise AssertionError(f"{what}: {int(bad.sum())} of {bad.size} elements outside {atol}+{rtol}*|ref|; worst at {i}: "
                             f"gpu={gpu[i]!r} ref={ref[i]!r}")
    return float((err / bound).max()) if err.size else 0.0


def run_and_check(w: W.Workload, rows=None, batched=False, scale=1.0, check_group=True):
    """Route -> group -> apply on the GPU, compare every step with the oracle.

    rows: optional token subset for the apply comparison (full-size configs); None = every row.
    Returns a dict of statistics (excluded gate tokens, worst error ratio)."""
    stats = {}
    r_ref, margin = oracle_route(w)
    r_dev = gpu_route(w)
    r_gpu = r_dev.cpu().numpy()
    keep = np.ones(w.N, dtype=bool)
    if margin is not None:
        keep = margin >= GATE_MARGIN
        stats["gate_excluded"] = int((~keep).sum())
        assert stats["gate_excluded"] <= max(4, int(0.01 * w.N)), "too many near-tie gate tokens"
    assert np.array_equal(r_gpu[keep], r_ref[keep]), "routing indices differ from the oracle"
    stats["gate_flipped"] = int((r_gpu != r_ref).sum())

    counts, offsets, perm = M.molora_group(r_dev, w.C)
    if check_group:
        c_ref, o_ref, p_ref = oracle.group(r_gpu, w.C)          # grouping of the routing the GPU produced: bit-exact
        assert np.array_equal(counts.cpu().numpy(), c_ref)
        assert np.array_equal(offsets.cpu().numpy(), o_ref)
        assert np.array_equal(perm.cpu().numpy()[: int(o_ref[-1])], p_ref)

    xs = {k: dev_tensor(v, w.dtype) for k, v in w.inputs.items()}
    ys = [dev_tensor(p.y, w.dtype) for p in w.projections]
    As = [dev_tensor(p.A, w.dtype) for p in w.projections]
    Bs = [dev_tensor(p.B, w.dtype) for p in w.projections]
    if batched:
        M.molora_apply_batched([M.ProjDesc(xs[p.x_key], y, A, B, scale) for p, y, A, B in
                                zip(w.projections, ys, As, Bs)], offsets, perm)
    else:
        for p, y, A, B in zip(w.projections, ys, As, Bs):
            M.molora_apply(xs[p.x_key], y, A, B, offsets, perm, scale=scale)
    torch.cuda.synchronize()

    sel = np.flatnonzero(keep) if rows is None else np.asarray([i for i in rows if keep[i]], dtype=np.int64)
    worst = 0.0
    for p, y in zip(w.projections, ys):
        ref = oracle.apply_rows(w.inputs[p.x_key], p.y, p.A, p.B, r_ref, sel, scale)
        got = to_f64(y[torch.from_numpy(sel).cuda()])
        worst = max(worst, assert_close(got, ref, what=f"{w.name}/{p.name}"))
        if w.dtype == "f32":
            assert_close(got, ref, ATOL32, RTOL32, what=f"{w.name}/{p.name} (fp32 bound)")
    stats["worst_ratio"] = worst
    return stats

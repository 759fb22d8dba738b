#!/usr/bin/env python
"""Benchmark of the routed-LoRA hot path (route -> group -> apply) on B200.

One "step" is one pass of the whole path over one batch of synthetic input.  The default workload is
the Qwen3-1.7B-shaped prefill configuration (N = 4096 tokens, q_proj 2048 -> 2048, bf16, C = 4 adapters
of rank 16, fp32 linear gate with top-1 argmax).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c5-iid] [--impl ours|reference]

N > 1 is launched with torch.distributed.run, one rank per GPU; every rank processes its own batches
(tokens are independent, Eq. 2: no collective on the data path; weak scaling) and the step time is
the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "routed_lora_tokens_per_s"
UNIT = "tokens/s"
L2_BYTES = 126e6
# dram__bytes_read.sum + dram__bytes_write.sum per apply launch from the committed ncu capture (profiles/), by workload
NCU_TRAFFIC_BYTES = {"c2": 34.17e6, "c3": 26.81e6, "c5": 615.3e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- workload description
def workload_info(w):
    """Algorithmic bytes / flops of one step's apply launch(es): x once + y read and written + the A_c, B_c
    of every adapter + perm/offsets; 2*N*rank*(d_in + d_out) flop (N token-adapter products, Theorem 3.6)."""
    e = 2 if w.dtype == "bf16" else 4
    by, fl = 0, 0
    for p in w.projections:
        by += w.N * p.d_in * e + 2 * w.N * p.d_out * e + w.C * p.rank * (p.d_in + p.d_out) * e
        fl += 2 * w.N * p.rank * (p.d_in + p.d_out)
    by += 4 * w.N + 4 * (w.C + 1)
    return by, fl


class Clocks(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.01):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz, self.ok = [], set(), None, False
        self._halt = threading.Event()
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception as exc:   # NVML missing: report that clocks could not be sampled
            self.err = repr(exc)

    NAMES = {0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
             0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
             0x100: "display_clock_setting"}

    def run(self):
        if not self.ok:
            return
        while not self._halt.is_set():
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
                bits = int(self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for b, name in self.NAMES.items():
                    if bits & b:
                        self.reasons.add(name)
            except Exception:
                pass
            self._halt.wait(self.period)

    def stop(self):
        self._halt.set()
        if self.is_alive():
            self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------- our arm
def build_sets(W, torch, name, n_sets, rank):
    """Device-resident buffer sets of the workload: shared weights, n_sets activation batches."""
    def dev(a, dtype):
        if a.dtype == np.int32:
            return torch.from_numpy(np.ascontiguousarray(a)).cuda()
        if dtype == "bf16":
            return torch.from_numpy(W.bf16_bits(a)).cuda().view(torch.bfloat16)
        return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()

    from paper_2603_15965_b200.shard import rank_batches
    batches = rank_batches(rank, max(1, int(os.environ.get("WORLD_SIZE", "1"))), n_sets)   # disjoint across ranks
    sets, w0 = [], None
    for b in range(n_sets):
        if name == "c2":
            w = W.get("c2", batch=batches[b])
        elif name == "c3":
            w = W.get("c3", layer=batches[b])
        else:
            w = W.get(name) if b == 0 else None
        if w is None:   # large configs: clone batch 0 into distinct buffers (same values, distinct addresses)
            s0 = sets[0]
            sets.append({"x": {k: v.clone() for k, v in s0["x"].items()}, "y": [t.clone() for t in s0["y"]],
                         "A": s0["A"], "B": s0["B"], "ids": s0["ids"], "r_given": s0["r_given"]})
            continue
        w0 = w0 or w
        weights_from = sets[0] if (sets and name == "c2") else None
        sets.append({
            "x": {k: dev(v, w.dtype) for k, v in w.inputs.items()},
            "y": [dev(p.y, w.dtype) for p in w.projections],
            "A": weights_from["A"] if weights_from else [dev(p.A, w.dtype) for p in w.projections],
            "B": weights_from["B"] if weights_from else [dev(p.B, w.dtype) for p in w.projections],
            "ids": dev(w.ids, "i") if w.ids is not None else None,
            "r_given": dev(w.r, "i") if w.r is not None else None,
        })
    gate_ws = None
    if w0.G is not None:
        import paper_2603_15965_b200 as M
        need = M.molora_route_gate_workspace_bytes(1 if w0.dtype == "bf16" else 0, w0.G.shape[0], w0.G.shape[1])
        gate_ws = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None
    shared = {"status": torch.zeros(1, dtype=torch.int32, device="cuda"), "gate_ws": gate_ws,
              "G": dev(w0.G, "f32") if w0.G is not None else None,
              "breaks": dev(w0.breaks, "i") if w0.breaks is not None else None}
    return w0, sets, shared


def marshal_step(lib, w, s, shared, stream_handle):
    """The step's three C-ABI calls as closures over already converted ctypes arguments (marshalling only)."""
    import ctypes
    from functools import partial
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    N, C = w.N, w.C
    st = vp(stream_handle)
    route = None
    if w.router == "gate":
        x = s["x"][w.gate_x_key]
        gws = shared["gate_ws"]
        route = partial(lib.molora_route_gate, vp(x.data_ptr()), 1 if w.dtype == "bf16" else 0, i64(N), i32(x.shape[1]),
                        i64(x.stride(0)), vp(shared["G"].data_ptr()), None, i32(C), vp(s["r"].data_ptr()), None,
                        vp(gws.data_ptr()) if gws is not None else None,
                        ctypes.c_size_t(gws.numel() if gws is not None else 0), st)
        r = s["r"]
    elif w.router == "vocab":
        route = partial(lib.molora_route_vocab, vp(s["ids"].data_ptr()), i64(N), vp(shared["breaks"].data_ptr()),
                        i32(shared["breaks"].numel() - 1), vp(s["r"].data_ptr()), None, st)
        r = s["r"]
    else:
        r = s["r_given"]
    group = partial(lib.molora_group, vp(r.data_ptr()), i64(N), i32(C), vp(s["counts"].data_ptr()),
                    vp(s["offsets"].data_ptr()), vp(s["perm"].data_ptr()), None, ctypes.c_size_t(0), None, st)
    arr, n, c, dt = s["packed"]
    aws = shared.get("apply_ws")
    apply = partial(lib.molora_apply_batched, arr, i32(len(arr)), dt, i64(n), i32(c), vp(s["offsets"].data_ptr()),
                    vp(s["perm"].data_ptr()), vp(aws.data_ptr()) if aws is not None else None,
                    ctypes.c_size_t(aws.numel() if aws is not None else 0), vp(shared["status"].data_ptr()), st)
    # the same two stages as ONE call (a single launch where the library can fuse them)
    group_apply = partial(lib.molora_group_apply_batched, vp(r.data_ptr()), i64(N), i32(C), vp(s["counts"].data_ptr()),
                          vp(s["offsets"].data_ptr()), vp(s["perm"].data_ptr()), arr, i32(len(arr)), dt,
                          vp(aws.data_ptr()) if aws is not None else None,
                          ctypes.c_size_t(aws.numel() if aws is not None else 0), vp(shared["status"].data_ptr()), st)
    return route, group, apply, group_apply


def run_ours(args):
    import torch
    import paper_2603_15965_b200 as M
    import paper_2603_15965_b200.binding  # noqa: F401
    from paper_2603_15965_b200 import shard
    from paper_2603_15965_b200 import workloads as W
    from paper_2603_15965_b200.binding import pack_proj_descs
    from paper_2603_15965_b200.build import build_library

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the routed-LoRA path has no CPU fallback")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build_library()
    if dist is not None:
        dist.barrier()
    lib = M.load_library()

    name = args.workload
    probe = W.get(name) if name != "c2" else W.get("c2", batch=0)
    step_bytes, step_flops = workload_info(probe)
    per_set = sum(v.nbytes // (2 if probe.dtype == "bf16" else 1) for v in probe.inputs.values()) + \
        sum(p.y.nbytes // (2 if probe.dtype == "bf16" else 1) for p in probe.projections)
    n_sets = max(2, int(np.ceil(2.5 * L2_BYTES / per_set)))          # rotation working set >= 2.5 x L2
    n_sets = min(n_sets, args.max_sets)
    del probe
    w, sets, shared = build_sets(W, torch, name, n_sets, rank)
    N, C = w.N, w.C
    stream = torch.cuda.Stream()      # every call of the timed region is enqueued (or captured) on this stream

    # per-set routing/grouping outputs (fixed addresses, as a serving stack would keep them)
    for s in sets:
        s["r"] = torch.empty(N, dtype=torch.int32, device="cuda")
        s["counts"] = torch.empty(C, dtype=torch.int32, device="cuda")
        s["offsets"] = torch.empty(C + 1, dtype=torch.int32, device="cuda")
        s["perm"] = torch.empty(N, dtype=torch.int32, device="cuda")
        s["packed"] = pack_proj_descs([M.ProjDesc(s["x"][p.x_key], y, A, B, 1.0) for p, y, A, B in
                                                 zip(w.projections, s["y"], s["A"], s["B"])])
    gate_launches = 0 if w.router == "given" else (2 if (w.router == "gate" and shared["gate_ws"] is not None) else 1)
    # scratch of the apply (partial shrink results of the two-launch small-tile path); one buffer serves every set
    from paper_2603_15965_b200.binding import molora_apply_batched_workspace_bytes
    need = molora_apply_batched_workspace_bytes(sets[0]["packed"][0], N, C)
    shared["apply_ws"] = torch.empty(need, dtype=torch.uint8, device="cuda") if need else None
    # launches of the apply: one per rank on the tensor-core path, shrink + expand on the small-tile path (which is the
    # one that asks for a workspace)
    apply_launches = sum(2 if any(M.molora_apply_workspace_bytes(N, C, p.d_in, p.d_out, p.rank) > 0
                                  for p in w.projections if p.rank == rk) else 1 for rk in {p.rank for p in w.projections})
    # grouping + apply are one C-ABI call; where the library fuses them (every projection on the streaming kernel or on
    # the two-launch kernels) the apply kernels group on chip, otherwise the grouping launch precedes the apply launches
    arr0, n0, c0, dt0 = sets[0]["packed"]
    fused = bool(lib.molora_group_apply_skips_group_launch(arr0, len(arr0), dt0, n0))   # grouping inside the apply kernels
    one_launch = bool(lib.molora_group_apply_is_one_launch(arr0, len(arr0), dt0, n0))
    launches_per_step = gate_launches + (1 if one_launch else apply_launches if fused else 1 + apply_launches)
    for s in sets:
        s["calls"] = marshal_step(lib, w, s, shared, stream.cuda_stream)

    def step(s, ev=None):
        """route -> group + apply on buffer set s: two C-ABI calls with pre-marshalled arguments."""
        route, group, apply, group_apply = s["calls"]
        if route is not None and route() != 0:
            raise RuntimeError("molora_route_* refused the call")
        if fused or ev is None:
            if ev is not None:
                ev[0].record(stream)
            if group_apply() != 0:
                raise RuntimeError("molora_group_apply_batched refused the call")
        else:
            # eager timing of a call the library does not fuse: the same two calls it makes, taken apart so that the
            # apply kernels can be bracketed by events
            if group() != 0:
                raise RuntimeError("molora_group refused the call")
            if ev is not None:
                ev[0].record(stream)
            if apply() != 0:
                raise RuntimeError("molora_apply_batched refused the call")
        if ev is not None:
            ev[1].record(stream)

    # ------------------------------------------------------------------ warm-up, then the timed region
    K = args.steps
    W0 = max(3, args.warmup)
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for i in range(W0):
            step(sets[i % n_sets])
        torch.cuda.synchronize()
        if args.launch == "graph":
            # The paper replays this path from a CUDA graph (fixed addresses, no host work between kernels); so does
            # the bench: K steps are captured in chunks and replayed, which removes the Python/driver launch cost
            # from a step that lasts tens of microseconds.  A second set of graphs holds only the apply calls over
            # the same buffer rotation; its replay time / K is the kernel time used for the roofline.
            CH = min(K, 512)

            def capture(fn, first, n):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    for k in range(first, first + n):
                        fn(sets[k % n_sets])
                return g

            reps, rem = divmod(K, CH)
            g_full, g_rem = capture(step, W0, CH), (capture(step, W0 + reps * CH, rem) if rem else None)
            kcall = 3 if fused else 2          # the dominant kernel: grouping + apply in one launch, or the apply
            a_full = capture(lambda s_: s_["calls"][kcall](), W0, CH)
            a_rem = capture(lambda s_: s_["calls"][kcall](), W0 + reps * CH, rem) if rem else None
            g_full.replay()
            torch.cuda.synchronize()
        clocks = Clocks(local)
        clocks.start()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        if args.launch == "graph":
            t0.record(stream)
            for _ in range(reps):
                g_full.replay()
            if g_rem is not None:
                g_rem.replay()
            t1.record(stream)
            torch.cuda.synchronize()
            total_ms = t0.elapsed_time(t1)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a0.record(stream)
            for _ in range(reps):
                a_full.replay()
            if a_rem is not None:
                a_rem.replay()
            a1.record(stream)
            torch.cuda.synchronize()
            apply_ms = a0.elapsed_time(a1) / K
            kernel_timing = "graphs of the dominant kernel's call alone over the same buffer rotation, CUDA events around K launches"
        else:
            ev_every = max(1, K // 2000)                               # bound the number of event pairs
            pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                     if k % ev_every == 0 else None for k in range(K)]
            t0.record(stream)
            for k in range(K):
                step(sets[(W0 + k) % n_sets], pairs[k])
            t1.record(stream)
            torch.cuda.synchronize()
            total_ms = t0.elapsed_time(t1)
            apply_ms = float(np.mean([a.elapsed_time(b) for p in pairs if p is not None for a, b in [p]]))
            kernel_timing = "CUDA event pair around every apply call (includes host launch gaps)"
        # latency of a single step replayed on its own (one graph per buffer set, one event pair per replay): the
        # distribution the paper reports for graph replay (median, P99, coefficient of variation)
        latency = None
        if args.launch == "graph" and not args.profile:
            singles = [capture(step, i, 1) for i in range(min(n_sets, 8))]
            n_lat = 400
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n_lat)]
            for i in range(16):
                singles[i % len(singles)].replay()
            torch.cuda.synchronize()
            for i, (e0, e1) in enumerate(evs):
                e0.record(stream)
                singles[i % len(singles)].replay()
                e1.record(stream)
            torch.cuda.synchronize()
            lat = np.sort(np.array([e0.elapsed_time(e1) * 1e3 for e0, e1 in evs]))
            latency = {"p50_us": float(lat[len(lat) // 2]), "p99_us": float(lat[int(len(lat) * 0.99) - 1]),
                       "cv": float(lat.std() / lat.mean()), "samples": n_lat,
                       "note": "one step per CUDA-graph replay, event pair around each replay (includes the graph launch)"}
        if dist is not None:
            dist.barrier()
        # keep the GPU busy a little longer (untimed) if the region was too short for the clock sampler
        t_end = time.time() + (0.25 if total_ms < 250 else 0.0)
        while time.time() < t_end:
            step(sets[0])
        torch.cuda.synchronize()
    clk = clocks.stop()

    total_ms = shard.max_over_ranks(total_ms, dist, device="cuda")     # the slowest rank defines the step
    ms_per_step = total_ms / K
    value = shard.aggregate_tokens_per_s(N, world, ms_per_step)

    # ------------------------------------------------------------------ end to end with host buffers
    e2e = None if args.profile else run_e2e(args, torch, M, w, sets, shared, world, dist)

    out = None
    if rank == 0:
        peaks = measured_peaks()
        achieved = step_bytes / (apply_ms * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "latency": latency, "n_gpus": world, "steps": K, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if w.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": f"{name}: N={N} tokens/GPU, C={C}, " + ", ".join(
                f"{p.name} {p.d_in}->{p.d_out} r{p.rank}" for p in w.projections) + f", router={w.router}",
                "tokens_per_step_per_gpu": N, "buffer_sets": n_sets,
                "l2": f"rotation over {n_sets} buffer sets ({n_sets * per_set / 1e6:.0f} MB > 126 MB L2)",
                "launch": ("CUDA graph replay of the C-ABI calls (route, then group + apply)" if args.launch == "graph"
                           else "eager, one C-ABI call per stage")},
            "gpu_launches": launches_per_step * K,
            "clocks": clk,
            "e2e": e2e,
            "roofline": {"bound": "hbm", "kernel": ("molora_group_apply_batched (grouping + grouped shrink+expand, no grouping launch)" if fused
                                                    else "molora_apply (grouped shrink+expand)"), "achieved": achieved,
                         "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                         "peak_source": peaks["source"], "traffic": NCU_TRAFFIC_BYTES.get(name),
                         "algorithmic_bytes": step_bytes, "kernel_ms": apply_ms, "kernel_timing": kernel_timing,
                         "algorithmic_tflops": step_flops / (apply_ms * 1e-3) / 1e12},
            "cpu_baseline": None if args.profile else cpu_baseline(name),
        }
    if dist is not None:
        dist.destroy_process_group()
    return out


def run_e2e(args, torch, M, w, sets, shared, world, dist):
    """Same metric through the host-buffer entry point: every step, molora_forward_host copies the step's
    activations (x, y; ids / r if routed from integers) from pinned host memory into a device arena, runs
    route -> group -> apply and copies h back to pinned host memory.  Two streams with one arena each alternate,
    so the copies of consecutive steps overlap (the PCIe link is full duplex)."""
    N, C = w.N, w.C
    s0 = sets[0]
    router = {"vocab": M.ROUTE_VOCAB, "gate": M.ROUTE_GATE, "given": M.ROUTE_GIVEN}[w.router]
    gate_proj = 0
    if w.router == "gate":
        gate_proj = [p.x_key for p in w.projections].index(w.gate_x_key)
    pristine = build_pristine_y(w, torch)
    lanes = []
    for _ in range(2):
        hx = {k: v.cpu().pin_memory() for k, v in s0["x"].items()}
        hy = [p.clone().pin_memory() for p in pristine]
        projs = [M.HostProj(hx[p.x_key], y, A, B, 1.0) for p, y, A, B in zip(w.projections, hy, s0["A"], s0["B"])]
        packed = M.binding.pack_host_projs(projs)
        arena = torch.empty(M.molora_forward_host_arena_bytes(None, router, gate_proj, packed=packed), dtype=torch.uint8,
                            device="cuda")
        src = None
        if w.router == "vocab":
            src = s0["ids"].cpu().pin_memory()
        elif w.router == "given":
            src = s0["r_given"].cpu().pin_memory()
        lanes.append({"hx": hx, "hy": hy, "packed": packed, "arena": arena, "src": src, "stream": torch.cuda.Stream()})
    h2d = sum(t.numel() * t.element_size() for t in list(lanes[0]["hx"].values()) + lanes[0]["hy"]) + \
        (lanes[0]["src"].numel() * 4 if lanes[0]["src"] is not None else 0)
    d2h = sum(t.numel() * t.element_size() for t in lanes[0]["hy"])

    def step(k):
        ln = lanes[k % 2]
        M.molora_forward_host(router, None, ln["arena"], route_src=ln["src"], breaks=shared["breaks"], G=shared["G"],
                              gate_proj=gate_proj, dev_status=shared["status"], stream=ln["stream"], packed=ln["packed"])

    K = max(4, min(args.steps, args.e2e_steps))
    for k in range(4):
        step(k)
    torch.cuda.synchronize()
    if dist is not None:
        dist.barrier()
    main = torch.cuda.current_stream()
    t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0.record(main)
    for ln in lanes:
        ln["stream"].wait_event(t0)
    for k in range(K):
        step(k)
    for ln in lanes:
        done = torch.cuda.Event()
        done.record(ln["stream"])
        main.wait_event(done)
    t1.record(main)
    torch.cuda.synchronize()
    ms = t0.elapsed_time(t1)
    if dist is not None:
        t = torch.tensor([ms], device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    return {"value": world * N / (ms / K * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "steps": K, "ms_per_step": ms / K,
            "note": "molora_forward_host: pinned host x, y (and ids / r) copied in, h copied out every step; "
                    "adapter and gate weights resident; two streams alternate"}


def build_pristine_y(w, torch):
    from paper_2603_15965_b200 import workloads as W
    out = []
    for p in w.projections:
        if w.dtype == "bf16":
            out.append(torch.from_numpy(W.bf16_bits(p.y)).view(torch.bfloat16))
        else:
            out.append(torch.from_numpy(p.y))
    return out


# ----------------------------------------------------------------------------- oracle legs (CPU)
def oracle_sample(name):
    """The bounded sample of the workload the oracle is timed on: (workload, description)."""
    from paper_2603_15965_b200 import workloads as W
    if name == "c2":
        return W.get("c2"), "the whole step: 4096 tokens, gate + group + apply"
    if name == "c3":
        return W.get("c3"), "the whole step: 256 tokens, group + 7 applies"
    if name == "c4":
        return W.get("c4", n_tokens=512), "512 of 8192 tokens, gate + group + 7 applies"
    if name.startswith("f9-") or name.startswith("t9-"):
        w = W.get(name)
        return w, f"the whole step: {w.N} tokens, group + apply"
    w = W.c5_multimodal(n_seqs=1, seq_len=2048, iid=name == "c5-iid")
    return w, "2048 of 16384 tokens (one sequence), vocab route + group + 2 applies"


def oracle_step(w):
    import oracle
    if w.router == "vocab":
        r = oracle.route_vocab(w.ids, w.breaks)
    elif w.router == "gate":
        r = oracle.route_gate(w.inputs[w.gate_x_key], w.G)[0]
    else:
        r = w.r
    oracle.group(r, w.C)
    for p in w.projections:
        oracle.apply(w.inputs[p.x_key], p.y, p.A, p.B, r)


def cpu_baseline(name, reps=3):
    import oracle
    w, sample = oracle_sample(name)
    oracle_step(w)                                             # page in
    best = min(_timed(oracle_step, w) for _ in range(reps))
    return {"value": w.N / best, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample,
            "seconds_per_sample": best}


def _timed(fn, *a):
    t = time.perf_counter()
    fn(*a)
    return time.perf_counter() - t


def run_reference(args):
    """The oracle, as it stands, on the host cores: same metric, config and unit as our arm."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return None
    w, sample = oracle_sample(args.workload)
    for _ in range(min(args.warmup, 2)):
        oracle_step(w)
    K = max(1, min(args.steps, 20))
    t = time.perf_counter()
    for _ in range(K):
        oracle_step(w)
    sec = (time.perf_counter() - t) / K
    value = w.N / sec
    return {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
            "warmup": min(args.warmup, 2), "ms_per_step": sec * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{args.workload}: CPU oracle on a bounded sample ({sample})"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=50)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    from paper_2603_15965_b200.workloads import SWEEP_NAMES
    ap.add_argument("--workload", default="c2", choices=["c2", "c3", "c4", "c5", "c5-iid", *SWEEP_NAMES],
                    help="c2 (default, the headline configuration) .. c5; f9-<N> / t9-<skew>: batch and skew sweeps")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="replay the timed steps from CUDA graphs (default) or launch them one by one")
    ap.add_argument("--max-sets", type=int, default=32)
    ap.add_argument("--e2e-steps", type=int, default=50)
    ap.add_argument("--profile", action="store_true",
                    help="timed steps only: skip the host-buffer e2e leg and the oracle leg (for ncu captures)")
    args = ap.parse_args()
    out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()

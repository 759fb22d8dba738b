#!/usr/bin/env python
"""Benchmark of the routed-LoRA hot path (route -> group -> apply) on B200.

One "step" is one pass of the whole path over one batch of synthetic input.  With no --workload the headline is the
largest single-GPU configuration, the Qwen3-8B-shaped prefill layer c4 (N = 8192 tokens, seven projections, bf16,
C = 16 adapters of rank 64, fp32 linear gate with top-1 argmax), and the same JSON line carries, under "configs",
the step time, dominant-kernel time, algorithmic bytes and roofline fraction of the other configurations
(c2, c3, c5, c5-iid; the two c5 records also time the K = 4-pass per-sequence baseline).  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2|c3|c4|c5|c5-iid|f9-*|t9-*|t6-*] [--impl ours|reference]

Timing does not depend on K: the K steps are captured into CUDA graphs over a rotation of buffer sets larger than
L2, and that K-step pass is replayed until the timed leg has lasted at least --min-leg-s seconds (0.3 by default);
every pass has its own CUDA-event pair and the reported step time is the median pass time / K.

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
HBM_SPEC_GBS = 8000.0          # the nominal figure the targets are stated against; the measured copy rate is the peak
HEADLINE = "c4"
SUB_CONFIGS = ("c2", "c3", "c5", "c5-iid")
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from the ncu captures summarised
# under profiles/ (file named per entry); None where no capture of that workload is committed
GATHER_RW_GBS = 5277.0        # microbench/gather_rw.cu on this machine's B200: gathered 128-byte pieces, 2 reads : 1 write
NCU_TRAFFIC = {
    "c2": (34.17e6, "profiles/apply_stream_c2_full.md"),
    "c3": (26.81e6, "profiles/apply_stream_c3_full.md"),
    "c4": (1875e6, "profiles/apply_umma_c4_full.md (dram__bytes_read + write of one launch at full size, a one-pass capture)"),
    "c5": (615.4e6, "profiles/apply_umma_c5_full.md"),
    "c5-iid": (615.4e6, "profiles/apply_umma_c5_full.md (the c5 capture: same bytes, another routing)"),
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ----------------------------------------------------------------------------- workload description
FULL_TOKENS = {"c2": 4096, "c3": 256, "c4": 8192, "c5": 16384, "c5-iid": 16384}


def workload_label(name, w):
    """The same description of a workload for both arms (the reference arm runs a bounded sample of it)."""
    n = FULL_TOKENS.get(name, w.N)
    return f"{name}: N={n} tokens/GPU, C={w.C}, " + ", ".join(
        f"{p.name} {p.d_in}->{p.d_out} r{p.rank}" for p in w.projections) + f", router={w.router}"


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
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

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
def build_sets(W, torch, name, n_sets, rank, kw=None):
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
            w = W.get("c2", batch=batches[b], **(kw or {}))
        elif name == "c3":
            w = W.get("c3", layer=batches[b], **(kw or {}))
        else:
            w = W.get(name, **(kw or {})) if b == 0 else None
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
    G_dev = dev(w0.G, "f32") if w0.G is not None else None
    if G_dev is not None:
        import paper_2603_15965_b200 as M
        gate_ws = M.molora_route_gate_prepare(torch.bfloat16 if w0.dtype == "bf16" else torch.float32, G_dev)
    shared = {"status": torch.zeros(1, dtype=torch.int32, device="cuda"), "gate_ws": gate_ws,
              "G": G_dev,
              "breaks": dev(w0.breaks, "i") if w0.breaks is not None else None}
    return w0, sets, shared


def marshal_step(lib, w, s, shared, stream_handle):
    """The step's C-ABI calls as closures over already converted ctypes arguments (marshalling only)."""
    import ctypes
    from functools import partial
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    N, C = w.N, w.C
    st = vp(stream_handle)
    route = None
    if w.router == "gate":
        x = s["x"][w.gate_x_key]
        gws = shared["gate_ws"]
        # the gate's weights are static: their three-term images were built once, outside the timed region
        # (molora_route_gate_prepare); gates that need no image (C <= 4) take the same call
        route = partial(lib.molora_route_gate_prepared, vp(x.data_ptr()), 1 if w.dtype == "bf16" else 0, i64(N), i32(x.shape[1]),
                        i64(x.stride(0)), vp(shared["G"].data_ptr()), None, i32(C), vp(s["r"].data_ptr()), None,
                        vp(gws.data_ptr()) if gws is not None else None,
                        ctypes.c_size_t(gws.numel() if gws is not None else 0), None, st)
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


def timed_passes(torch, stream, run_pass, min_leg_s, max_passes=100000):
    """Replay `run_pass(i)` (which enqueues one K-step pass on `stream`) until the leg has lasted min_leg_s seconds of
    device time; one event pair per pass.  Returns the per-pass times in ms."""
    def batch(first, n):
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(n)]
        for j, (a, b) in enumerate(evs):
            a.record(stream)
            run_pass(first + j)
            b.record(stream)
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in evs]

    times = batch(0, 2)
    while sum(times) < min_leg_s * 1e3 and len(times) < max_passes:
        per = max(1e-4, float(np.median(times)))
        todo = int(min(max_passes - len(times), max(1, np.ceil((min_leg_s * 1e3 - sum(times)) / per * 1.05)), 4096))
        times += batch(len(times), todo)
    return times


def measure(name, args, env, headline):
    """Builds the buffer sets of workload `name`, runs warm-up, the timed step leg, the dominant-kernel leg and (c5) the
    K-pass baseline leg; returns the record of the workload."""
    torch, M, lib, W, shard, dist = env["torch"], env["M"], env["lib"], env["W"], env["shard"], env["dist"]
    rank, world, local = env["rank"], env["world"], env["local"]
    from paper_2603_15965_b200.binding import molora_apply_batched_workspace_bytes, pack_proj_descs

    # --tokens shrinks c2 / c3 / c4 (for profiler captures, which must stay small); never used for a reported number
    kw = {"n_tokens": args.tokens} if args.tokens and name in ("c2", "c3", "c4") else {}
    probe = W.get(name, **kw) if name != "c2" else W.get("c2", batch=0, **kw)
    step_bytes, step_flops = workload_info(probe)
    esz = 2 if probe.dtype == "bf16" else 1
    per_set = sum(v.nbytes // esz for v in probe.inputs.values()) + sum(p.y.nbytes // esz for p in probe.projections)
    n_sets = max(2, int(np.ceil(2.5 * L2_BYTES / per_set)))          # rotation working set >= 2.5 x L2
    n_sets = min(n_sets, args.max_sets)
    del probe
    w, sets, shared = build_sets(W, torch, name, n_sets, rank, kw)
    N, C = w.N, w.C
    stream = torch.cuda.Stream()      # every call of the timed region is enqueued (or captured) on this stream

    # per-set routing/grouping outputs (fixed addresses, as a serving stack would keep them)
    for i, s in enumerate(sets):
        s["idx"] = i
        s["r"] = torch.empty(N, dtype=torch.int32, device="cuda")
        s["counts"] = torch.empty(C, dtype=torch.int32, device="cuda")
        s["offsets"] = torch.empty(C + 1, dtype=torch.int32, device="cuda")
        s["perm"] = torch.empty(N, dtype=torch.int32, device="cuda")
        s["packed"] = pack_proj_descs([M.ProjDesc(s["x"][p.x_key], y, A, B, 1.0) for p, y, A, B in
                                       zip(w.projections, s["y"], s["A"], s["B"])])
    # scratch of the apply; one buffer serves every set (zero-filled: the kernels that keep counters there expect that
    # on first use and leave it so)
    need = molora_apply_batched_workspace_bytes(sets[0]["packed"][0], N, C)
    shared["apply_ws"] = torch.zeros(need, dtype=torch.uint8, device="cuda") if need else None
    arr0, n0, c0, dt0 = sets[0]["packed"]
    fused = bool(lib.molora_group_apply_skips_group_launch(arr0, len(arr0), dt0, n0, c0))   # grouping inside the apply kernels
    for s in sets:
        s["calls"] = marshal_step(lib, w, s, shared, stream.cuda_stream)

    def step(s):
        """route -> group + apply on buffer set s: two C-ABI calls with pre-marshalled arguments."""
        route, group, apply, group_apply = s["calls"]
        if route is not None and route() != 0:
            raise RuntimeError("molora_route_* refused the call")
        if group_apply() != 0:
            raise RuntimeError("molora_group_apply_batched refused the call")

    def checked(call):
        def f(s_):
            if call(s_) != 0:
                raise RuntimeError("a molora_* call was refused")
        return f

    K = args.steps
    W0 = max(3, args.warmup)
    rec = {}
    kcall = 3 if fused else 2          # the dominant kernel: grouping + apply in one call, or the apply
    with torch.cuda.stream(stream):
        # launches of a step and of the dominant kernel's call, counted by the library while the warm-up steps run
        n0 = M.molora_launch_count()
        step(sets[0])
        launches_per_step = M.molora_launch_count() - n0
        n0 = M.molora_launch_count()
        if sets[0]["calls"][kcall]() != 0:
            raise RuntimeError("the dominant kernel's call was refused")
        kernel_launches = M.molora_launch_count() - n0
        for i in range(W0):
            step(sets[i % n_sets])
        torch.cuda.synchronize()
        CH = min(K, 512)

        def capture(fn, first, n):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=stream):
                for k in range(first, first + n):
                    fn(sets[k % n_sets])
            return g

        def capture_pass(fn, first):
            """Graphs that together hold K consecutive steps of the rotation starting at step `first`."""
            reps, rem = divmod(K, CH)
            gs = [capture(fn, first, CH)] * reps          # the chunk graph is replayed `reps` times
            if rem:
                gs.append(capture(fn, first + reps * CH, rem))
            return gs

        # variants of the pass that start at different points of the rotation, so that a pass shorter than the
        # rotation still sees every buffer set cold
        n_var = 1 if args.launch == "eager" else max(1, min(8, int(np.ceil(n_sets / K))))
        if args.launch == "graph":
            step_graphs = [capture_pass(step, W0 + v * K) for v in range(n_var)]
            kern_graphs = [capture_pass(checked(lambda s_: s_["calls"][kcall]()), W0 + v * K) for v in range(n_var)]
            for gs in step_graphs:
                for g in gs:
                    g.replay()
            torch.cuda.synchronize()

            def step_pass(i):
                for g in step_graphs[i % n_var]:
                    g.replay()

            def kern_pass(i):
                for g in kern_graphs[i % n_var]:
                    g.replay()
            kernel_timing = ("graphs of the dominant kernel's call alone over the same buffer rotation; CUDA events around "
                             "each K-launch pass, median pass / K")
        else:
            def step_pass(i):
                for k in range(K):
                    step(sets[(W0 + i * K + k) % n_sets])

            def kern_pass(i):
                for k in range(K):
                    sets[(W0 + i * K + k) % n_sets]["calls"][kcall]()
            kernel_timing = "eager launches of the dominant kernel's call; CUDA events around each K-launch pass (includes host launch gaps)"

        clocks = Clocks(local)
        clocks.start()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        step_times = timed_passes(torch, stream, step_pass, args.min_leg_s)
        if dist is not None:
            dist.barrier()
        kern_times = timed_passes(torch, stream, kern_pass, args.min_leg_s)
        clk = clocks.stop()
        ms_per_step = shard.max_over_ranks(float(np.median(step_times)) / K, dist, device="cuda")   # slowest rank
        apply_ms = float(np.median(kern_times)) / K
        rec["passes"] = {"step": len(step_times), "kernel": len(kern_times),
                         "timed_region_s": (sum(step_times) + sum(kern_times)) * 1e-3, "pass_variants": n_var}

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

        kpass = None
        if name.startswith(("c5", "t6-")) and not args.profile and args.launch == "graph":
            kpass = run_kpass(args, env, w, sets, shared, stream, capture_pass, apply_ms, K, n_var)
        torch.cuda.synchronize()
        # every kernel of the timed region ORs what it detects into one status word: a bounded wait that gave up (or a
        # routing value out of range) would make the timing meaningless
        dev_status = int(shared["status"].item())
        if dev_status != 0:
            raise RuntimeError(f"device status word after the timed region: {dev_status:#x}")

    peaks = measured_peaks()
    achieved = step_bytes / (apply_ms * 1e-3) / 1e9
    traffic = NCU_TRAFFIC.get(name)
    rec.update({
        "workload": workload_label(name, w) + (f" [REDUCED to {w.N} tokens for a profiler capture]" if kw else ""),
        "tokens_per_step_per_gpu": N, "buffer_sets": n_sets,
        "l2": f"rotation over {n_sets} buffer sets ({n_sets * per_set / 1e6:.0f} MB > 126 MB L2)",
        "value": shard.aggregate_tokens_per_s(N, world, ms_per_step), "ms_per_step": ms_per_step,
        "launches_per_step": launches_per_step, "latency": latency, "clocks": clk, "dtype": "bf16" if w.dtype == "bf16" else "f32",
        "roofline": {"bound": "hbm",
                     "kernel": ("molora_group_apply_batched (grouping + grouped shrink+expand, no grouping launch)" if fused
                                else "molora_apply_batched (grouped shrink+expand)"),
                     "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"],
                     "peak_source": peaks["source"], "frac_of_spec": achieved / HBM_SPEC_GBS, "spec_gbs": HBM_SPEC_GBS,
                     "traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None,
                     "algorithmic_bytes": step_bytes, "kernel_ms": apply_ms, "kernel_launches": kernel_launches,
                     "kernel_timing": kernel_timing, "algorithmic_tflops": step_flops / (apply_ms * 1e-3) / 1e12},
    })
    if traffic and name in ("c4", "c5", "c5-iid") and not kw:
        # the measured DRAM traffic of the launch against what a do-nothing kernel with the same access pattern (gathered
        # 128-byte row pieces, 2 reads : 1 write) gets out of DRAM; context for `frac`, whose denominator is a sequential copy
        rate = traffic[0] / (apply_ms * 1e-3) / 1e9
        rec["roofline"]["traffic_rate_gbs"] = rate
        rec["roofline"]["pattern_ceiling"] = {"gbs": GATHER_RW_GBS, "frac": rate / GATHER_RW_GBS,
                                              "source": "profiles/gather_pattern_microbench.md"}
    if kpass is not None:
        rec["kpass_baseline"] = kpass
    rec["e2e"] = None
    if headline and not args.profile:
        rec["e2e"] = run_e2e(args, torch, M, w, sets, shared, world, dist)
    del sets, shared
    torch.cuda.empty_cache()
    return rec


def run_kpass(args, env, w, sets, shared, stream, capture_pass, single_ms, K, n_var):
    """The per-sequence baseline on the same kernels (Theorem 3.6): K_ad = C passes, pass k applies adapter k to ALL N
    tokens into its own copy of y (constant routing: offsets / perm are prepared once, no grouping inside the timed
    region), then one row select keeps, for every token, the row of the pass of its own adapter.  Timed like the step."""
    torch, lib = env["torch"], env["lib"]
    import ctypes
    from functools import partial
    import paper_2603_15965_b200 as M
    from paper_2603_15965_b200.binding import pack_proj_descs
    vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
    N, C = w.N, w.C
    ident = torch.arange(N, dtype=torch.int32, device="cuda")
    offs = []
    for k in range(C):
        o = torch.zeros(C + 1, dtype=torch.int32, device="cuda")
        o[k + 1:] = N
        offs.append(o)
    aws = shared.get("apply_ws")
    st = vp(stream.cuda_stream)
    # two scratch sets (> 2.5 x L2 together): [C, N, d_out] per projection, pre-filled with y = xW
    kp_sets = []
    for s in sets[:2]:
        stacks = [y.unsqueeze(0).repeat(C, 1, 1).contiguous() for y in s["y"]]
        outs = [torch.empty_like(y) for y in s["y"]]
        calls = []
        for k in range(C):
            packed = pack_proj_descs([M.ProjDesc(s["x"][p.x_key], stk[k], A, B, 1.0) for p, stk, A, B in
                                      zip(w.projections, stacks, s["A"], s["B"])])
            arr, n, c, dt = packed
            calls.append((packed, partial(lib.molora_apply_batched, arr, i32(len(arr)), dt, i64(n), i32(c),
                                          vp(offs[k].data_ptr()), vp(ident.data_ptr()),
                                          vp(aws.data_ptr()) if aws is not None else None,
                                          ctypes.c_size_t(aws.numel() if aws is not None else 0),
                                          vp(shared["status"].data_ptr()), st)))
        rsel = s["r" if w.router != "given" else "r_given"].to(torch.int64).clamp_(min=0) * N + torch.arange(N, device="cuda")
        kp_sets.append({"stacks": stacks, "outs": outs, "calls": calls, "rsel": rsel})

    def kpass_step(s):
        ks = kp_sets[s["idx"] % len(kp_sets)]
        rsel = ks["rsel"]
        for _, call in ks["calls"]:
            if call() != 0:
                raise RuntimeError("molora_apply_batched refused a pass of the K-pass baseline")
        for stk, out in zip(ks["stacks"], ks["outs"]):
            torch.index_select(stk.view(C * N, -1), 0, rsel, out=out)

    graphs = [capture_pass(kpass_step, v * K) for v in range(n_var)]

    def kp_pass(i):
        for g in graphs[i % n_var]:
            g.replay()
    kp_pass(0)
    torch.cuda.synchronize()
    times = timed_passes(torch, stream, kp_pass, args.min_leg_s)
    kp_ms = float(np.median(times)) / K
    return {"K": C, "kpass_ms": kp_ms, "single_pass_ms": single_ms, "ratio": kp_ms / single_ms,
            "token_adapter_products": {"single_pass": N, "kpass": C * N},
            "note": "K applies with constant routing over all N tokens into K copies of y + one row select, against the "
                    "single grouped pass (the dominant-kernel leg); same kernels, same buffer rotation, CUDA-graph replay"}


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
        arena = torch.zeros(M.molora_forward_host_arena_bytes(None, router, gate_proj, packed=packed), dtype=torch.uint8,
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


def run_ours(args):
    import torch
    import paper_2603_15965_b200 as M
    import paper_2603_15965_b200.binding  # noqa: F401
    from paper_2603_15965_b200 import shard
    from paper_2603_15965_b200 import workloads as W
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
    env = {"torch": torch, "M": M, "lib": M.load_library(), "W": W, "shard": shard, "dist": dist, "rank": rank,
           "world": world, "local": local}

    name = args.workload or HEADLINE
    head = measure(name, args, env, headline=True)
    subs = {}
    if args.workload is None and not args.profile:
        for sub in SUB_CONFIGS:
            subs[sub] = measure(sub, args, env, headline=False)

    out = None
    if rank == 0:
        K = args.steps
        passes = head["passes"]["step"]
        out = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "latency": head["latency"], "n_gpus": world, "steps": K,
            "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic",
            "config": {"workload": head["workload"], "tokens_per_step_per_gpu": head["tokens_per_step_per_gpu"],
                       "buffer_sets": head["buffer_sets"], "l2": head["l2"],
                       "launch": ("CUDA graph replay of the C-ABI calls (route, then group + apply)" if args.launch == "graph"
                                  else "eager, one C-ABI call per stage"),
                       "timing": f"the K-step pass is replayed until the leg lasts >= {args.min_leg_s} s; one CUDA-event pair "
                                 f"per pass; ms_per_step = median pass / K ({passes} passes here)"},
            "gpu_launches": head["launches_per_step"] * K * passes, "gpu_launches_per_step": head["launches_per_step"],
            "passes": head["passes"], "clocks": head["clocks"], "e2e": head["e2e"], "roofline": head["roofline"],
            "cpu_baseline": None if args.profile else cpu_baseline(name),
        }
        if head.get("kpass_baseline") is not None:
            out["kpass_baseline"] = head["kpass_baseline"]
        if subs:
            out["configs"] = {k: {"workload": v["workload"], "tokens_per_s": v["value"], "ms_per_step": v["ms_per_step"],
                                  "kernel_ms": v["roofline"]["kernel_ms"], "kernel": v["roofline"]["kernel"],
                                  "algorithmic_bytes": v["roofline"]["algorithmic_bytes"],
                                  "achieved_gbs": v["roofline"]["achieved"], "frac": v["roofline"]["frac"],
                                  "frac_of_spec": v["roofline"]["frac_of_spec"], "traffic": v["roofline"]["traffic"],
                                  "launches_per_step": v["launches_per_step"], "buffer_sets": v["buffer_sets"],
                                  "passes": v["passes"], "clocks": v["clocks"], "latency": v["latency"],
                                  **({"kpass_baseline": v["kpass_baseline"]} if v.get("kpass_baseline") else {})}
                              for k, v in subs.items()}
    if dist is not None:
        dist.destroy_process_group()
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
    if name.startswith(("f9-", "t9-", "t6-")):
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
    name = args.workload or HEADLINE
    w, sample = oracle_sample(name)
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
            "config": {"workload": workload_label(name, w), "sample": f"CPU oracle on a bounded sample: {sample}"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    from paper_2603_15965_b200.workloads import SWEEP_NAMES
    ap.add_argument("--workload", default=None, choices=["c2", "c3", "c4", "c5", "c5-iid", *SWEEP_NAMES],
                    help="default: c4 as the headline plus sub-records of c2, c3, c5, c5-iid; "
                         "f9-<N> / t9-<skew> / t6-<distribution>: batch, skew and modality-distribution sweeps")
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="replay the timed steps from CUDA graphs (default) or launch them one by one")
    ap.add_argument("--min-leg-s", type=float, default=0.3, help="every timed leg lasts at least this long")
    ap.add_argument("--max-sets", type=int, default=32)
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--tokens", type=int, default=0,
                    help="profiler captures only: run c2 / c3 / c4 with this many tokens instead of the configuration's")
    ap.add_argument("--profile", action="store_true",
                    help="timed steps of one workload only: no sub-records, no host-buffer e2e leg, no oracle leg (for ncu captures)")
    args = ap.parse_args()
    out = run_reference(args) if args.impl == "reference" else run_ours(args)
    if out is not None:
        print(json.dumps(out))


if __name__ == "__main__":
    main()

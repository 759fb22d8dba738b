"""Seeded synthetic inputs for the routed-LoRA path (shapes of the five benchmark configurations).

This module only *draws inputs*: token ids, routing sources, activations, adapter stacks and gate
weights, with the shapes and value distributions of the workloads.  It contains none of the method's
arithmetic (no routing, grouping, shrink or expand) and is the one module that both the CPU oracle's
tests and the CUDA path's tests/bench import, so that both sides see bit-identical inputs.

Conventions
-----------
* Every tensor is returned as a numpy ``float32`` (or ``int32``) array.  For bf16 workloads the
  values are rounded to bf16 (round-to-nearest-even) once, here, so the fp32 array holds exactly
  bf16-representable numbers; :func:`bf16_bits` gives the 16-bit patterns to upload.
* ``N(0, v)`` in the workload descriptions is read with ``v`` the **variance**:
  sigma_A = d_in**-0.5, sigma_W = sigma_G = d**-0.5, sigma_B = 0.1.
* Generator: configuration ``cfg`` owns ``SeedSequence(260315965).spawn(9)[cfg]``; its child stream 0 draws
  the routing source and the weights (ids / r, A, B per projection, G, in that order) and child stream
  ``1 + b`` draws activation batch ``b`` (x*, then y* / W), so weights do not depend on the token count.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional

import numpy as np

ROOT_SEED = 260315965


# ----------------------------------------------------------------------------- bf16 helpers
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round an fp32 array to the nearest bf16 value (ties to even); result stays fp32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    out = ((u + bias) & np.uint32(0xFFFF0000)).view(np.float32)
    return out.reshape(a.shape)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """16-bit patterns (as int16) of an fp32 array that already holds bf16-representable values."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    if np.any(u & np.uint32(0xFFFF)):
        raise ValueError("array is not bf16-representable; call round_to_bf16 first")
    return (u >> np.uint32(16)).astype(np.uint16).view(np.int16).reshape(a.shape)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    """Inverse of :func:`bf16_bits`: int16/uint16 patterns -> fp32 values."""
    u = np.ascontiguousarray(bits).view(np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).reshape(bits.shape)


# ----------------------------------------------------------------------------- containers
@dataclass
class Projection:
    """One adapted projection d_in -> d_out: reads activations ``inputs[x_key]``, updates ``y`` in place."""
    name: str
    x_key: str
    d_in: int
    d_out: int
    rank: int
    A: np.ndarray          # [C, d_in, rank]
    B: np.ndarray          # [C, rank, d_out]
    y: np.ndarray          # [N, d_out]  base projection output x W (caller-provided)


@dataclass
class Workload:
    name: str
    N: int
    C: int
    dtype: str                       # "f32" | "bf16": storage type of x, y, A, B
    router: str                      # "vocab" | "gate" | "given"
    inputs: Dict[str, np.ndarray]    # activations by key, each [N, d]
    projections: List[Projection]
    scale: float = 1.0
    ids: Optional[np.ndarray] = None       # int32 [N]            (router == "vocab")
    breaks: Optional[np.ndarray] = None    # int32 [M+1]          (router == "vocab")
    G: Optional[np.ndarray] = None         # fp32 [d, C]          (router == "gate")
    gate_x_key: Optional[str] = None       # activations the gate reads
    r: Optional[np.ndarray] = None         # int32 [N]            (router == "given")
    seq_id: Optional[np.ndarray] = None    # int32 [N] sequence membership (context only)
    notes: Dict[str, object] = field(default_factory=dict)


def _rng(cfg_index: int, stream: int) -> np.random.Generator:
    """Child stream ``stream`` of configuration ``cfg_index`` (0 = routing source + weights, 1+b = batch b)."""
    ss = np.random.SeedSequence(ROOT_SEED).spawn(9)[cfg_index]      # children 0..4: c1..c5; 6, 7, 8: the sweeps
    return np.random.default_rng(ss.spawn(stream + 1)[stream])


def _normal(rng, shape, sigma, bf16):
    a = rng.standard_normal(shape, dtype=np.float32)
    if sigma != 1.0:
        a *= np.float32(sigma)
    return round_to_bf16(a) if bf16 else a


def _adapters(rng, C, d_in, d_out, rank, bf16):
    A = _normal(rng, (C, d_in, rank), d_in ** -0.5, bf16)
    B = _normal(rng, (C, rank, d_out), 0.1, bf16)
    return A, B


# ----------------------------------------------------------------------------- c1
def c1_tiny_vocab() -> Workload:
    """N=256 (2 x 128), ids uniform in [0,2000), ids<1000 -> adapter 0, else 1; fp32, 512->512, rank 8."""
    wrng, rng = _rng(0, 0), _rng(0, 1)
    N, d, rank, C = 256, 512, 8, 2
    ids = wrng.integers(0, 2000, size=N, dtype=np.int32)
    A, B = _adapters(wrng, C, d, d, rank, False)
    x = _normal(rng, (N, d), 1.0, False)
    W = _normal(rng, (d, d), d ** -0.5, False)
    y = (x.astype(np.float64) @ W.astype(np.float64)).astype(np.float32)   # base projection, outside the path
    return Workload(
        name="c1", N=N, C=C, dtype="f32", router="vocab", inputs={"x": x},
        projections=[Projection("proj", "x", d, d, rank, A, B, y)],
        ids=ids, breaks=np.array([0, 1000, 2000], dtype=np.int32),
        seq_id=np.repeat(np.arange(2, dtype=np.int32), 128), notes={"W": W})


# ----------------------------------------------------------------------------- c2
def c2_prefill_1p7b(n_tokens: int = 4096, batch: int = 0) -> Workload:
    """Qwen3-1.7B-shaped prefill, one q_proj 2048->2048, bf16, C=4 rank 16, fp32 linear gate 2048x4.

    ``batch`` selects the activation batch (x, y); adapters and gate are the same for every batch."""
    wrng, rng = _rng(1, 0), _rng(1, 1 + batch)
    N, d, rank, C = n_tokens, 2048, 16, 4
    A, B = _adapters(wrng, C, d, d, rank, True)
    G = _normal(wrng, (d, C), d ** -0.5, False)
    x = _normal(rng, (N, d), 1.0, True)
    y = _normal(rng, (N, d), 1.0, True)
    return Workload(
        name="c2", N=N, C=C, dtype="bf16", router="gate", inputs={"x": x},
        projections=[Projection("q_proj", "x", d, d, rank, A, B, y)],
        G=G, gate_x_key="x", seq_id=np.repeat(np.arange(max(1, N // 1024), dtype=np.int32), min(N, 1024))[:N])


# ----------------------------------------------------------------------------- c3 / c4: one layer, 7 projections
def _layer(wrng, rng, N, C, hidden, kv, inter, rank, bf16=True):
    inputs = {
        "x_attn": _normal(rng, (N, hidden), 1.0, bf16),
        "x_o": _normal(rng, (N, hidden), 1.0, bf16),
        "x_mlp": _normal(rng, (N, hidden), 1.0, bf16),
        "x_down": _normal(rng, (N, inter), 1.0, bf16),
    }
    shapes = [("q_proj", "x_attn", hidden, hidden), ("k_proj", "x_attn", hidden, kv),
              ("v_proj", "x_attn", hidden, kv), ("o_proj", "x_o", hidden, hidden),
              ("gate_proj", "x_mlp", hidden, inter), ("up_proj", "x_mlp", hidden, inter),
              ("down_proj", "x_down", inter, hidden)]
    ys = [_normal(rng, (N, do), 1.0, bf16) for (_, _, _, do) in shapes]
    projs = []
    for (name, key, di, do), y in zip(shapes, ys):
        A, B = _adapters(wrng, C, di, do, rank, bf16)
        projs.append(Projection(name, key, di, do, rank, A, B, y))
    return inputs, projs


def zipf_probs(C: int, s: float = 1.1) -> np.ndarray:
    p = np.arange(1, C + 1, dtype=np.float64) ** (-s)
    return p / p.sum()


def c3_decode_1p7b(layer: int = 0, n_tokens: int = 256) -> Workload:
    """Qwen3-1.7B-shaped decode: 256 sequences x 1 token, 7 projections of one layer, C=8 rank 16, Zipf(1.1) adapters.

    ``layer`` selects one of the independent layer buffer sets (same routing, fresh tensors)."""
    N, C = n_tokens, 8
    r = _rng(2, 0).choice(C, size=N, p=zipf_probs(C, 1.1)).astype(np.int32)
    # every layer owns its weights and activations: streams 1+2*layer (weights) and 2+2*layer (activations)
    inputs, projs = _layer(_rng(2, 1 + 2 * layer), _rng(2, 2 + 2 * layer), N, C, 2048, 1024, 6144, 16)
    return Workload(name="c3", N=N, C=C, dtype="bf16", router="given", inputs=inputs, projections=projs,
                    r=r, seq_id=np.arange(N, dtype=np.int32), notes={"layer": layer})


def c4_prefill_8b(n_tokens: int = 8192) -> Workload:
    """Qwen3-8B-shaped prefill: N=8192 (8 x 1024), 7 projections, C=16 rank 64, fp32 linear gate 4096x16."""
    wrng, rng = _rng(3, 0), _rng(3, 1)
    N, C = n_tokens, 16
    G = _normal(wrng, (4096, C), 4096 ** -0.5, False)
    inputs, projs = _layer(wrng, rng, N, C, 4096, 1024, 12288, 64)
    return Workload(name="c4", N=N, C=C, dtype="bf16", router="gate", inputs=inputs, projections=projs,
                    G=G, gate_x_key="x_attn",
                    seq_id=np.repeat(np.arange(max(1, N // 1024), dtype=np.int32), min(N, 1024))[:N])


# ----------------------------------------------------------------------------- c5
C5_BREAKS = np.array([0, 131072, 147456, 155648, 163840], dtype=np.int32)   # text / image / audio / video


def c5_modalities(rng, n_seqs: int, seq_len: int, M: int = 4, mean_run: int = 64, iid: bool = False) -> np.ndarray:
    """Modality index per token: runs with Geometric(1/mean_run) length (support >= 1), or iid uniform."""
    if iid:
        return rng.integers(0, M, size=n_seqs * seq_len, dtype=np.int32)
    out = np.empty(n_seqs * seq_len, dtype=np.int32)
    for s in range(n_seqs):
        pos, m = 0, int(rng.integers(0, M))
        while pos < seq_len:
            run = int(rng.geometric(1.0 / mean_run))
            out[s * seq_len + pos: s * seq_len + min(seq_len, pos + run)] = m
            pos += run
            m = (m + 1 + int(rng.integers(0, M - 1))) % M      # uniform over the other M-1 modalities
    return out


def c5_multimodal(n_seqs: int = 8, seq_len: int = 2048, iid: bool = False) -> Workload:
    """Interleaved multimodal, vocab-routed: N=16384 (8 x 2048), C=4 over a 160k vocab, 2048->2048 and 2048->6144, rank 32."""
    wrng, rng = _rng(4, 0), _rng(4, 2 if iid else 1)
    N, C, d, rank = n_seqs * seq_len, 4, 2048, 32
    mod = c5_modalities(rng, n_seqs, seq_len, C, 64, iid)
    lo = C5_BREAKS[:-1][mod].astype(np.int64)
    hi = C5_BREAKS[1:][mod].astype(np.int64)
    ids = (lo + (rng.random(N) * (hi - lo)).astype(np.int64)).astype(np.int32)
    x = _normal(rng, (N, d), 1.0, True)
    projs = []
    ys = [_normal(rng, (N, do), 1.0, True) for do in (2048, 6144)]
    for name, do, y in zip(("proj_2048", "proj_6144"), (2048, 6144), ys):
        A, B = _adapters(wrng, C, d, do, rank, True)
        projs.append(Projection(name, "x", d, do, rank, A, B, y))
    return Workload(name="c5-iid" if iid else "c5", N=N, C=C, dtype="bf16", router="vocab", inputs={"x": x},
                    projections=projs, ids=ids, breaks=C5_BREAKS.copy(),
                    seq_id=np.repeat(np.arange(n_seqs, dtype=np.int32), seq_len), notes={"modality": mod})


# ----------------------------------------------------------------------------- free-form problems for edge tests
def random_problem(seed: int, N: int, C: int, d_in: int, d_out: int, rank: int, dtype: str = "bf16",
                   r: Optional[np.ndarray] = None, unrouted_frac: float = 0.0, sigma_b: float = 0.1) -> Workload:
    """A single projection with a given (or uniform random) routing vector; used by edge-shape tests."""
    rng = np.random.default_rng(np.random.SeedSequence([ROOT_SEED, seed]))
    bf16 = dtype == "bf16"
    if r is None:
        r = rng.integers(0, C, size=N, dtype=np.int32)
        if unrouted_frac > 0:
            r[rng.random(N) < unrouted_frac] = -1
    r = np.asarray(r, dtype=np.int32)
    x = _normal(rng, (N, d_in), 1.0, bf16)
    y = _normal(rng, (N, d_out), 1.0, bf16)
    A = _normal(rng, (C, d_in, rank), d_in ** -0.5, bf16)
    B = _normal(rng, (C, rank, d_out), sigma_b, bf16)
    return Workload(name=f"rand{seed}", N=N, C=C, dtype=dtype, router="given", inputs={"x": x},
                    projections=[Projection("proj", "x", d_in, d_out, rank, A, B, y)], r=r)


def segment_sizes_routing(sizes) -> np.ndarray:
    """Routing vector whose adapter c owns exactly sizes[c] tokens, interleaved round-robin (not pre-sorted)."""
    sizes = list(sizes)
    left = sizes[:]
    out = []
    while any(left):
        for c in range(len(sizes)):
            if left[c]:
                out.append(c)
                left[c] -= 1
    return np.asarray(out, dtype=np.int32)


# ----------------------------------------------------------------------------- sweeps (Figure 9, Table 9 conditions)
F9_BATCHES = (64, 128, 256, 512, 1024, 2048)
T9_SKEWS = {"uniform": (0.25, 0.25, 0.25, 0.25), "80": (0.80, 0.10, 0.05, 0.05), "95": (0.95, 0.02, 0.02, 0.01)}


def f9_batch(n_tokens: int) -> Workload:
    """Batch sweep at the conditions of the paper's kernel study (Figure 9): one projection 4096->4096, rank 64,
    8 adapters chosen uniformly at random, bf16; n_tokens in F9_BATCHES locates the crossover between the
    small-tile and the tensor-core path."""
    wrng, rng = _rng(7, 0), _rng(7, 1 + (F9_BATCHES.index(n_tokens) if n_tokens in F9_BATCHES else len(F9_BATCHES)))
    N, C, d, rank = n_tokens, 8, 4096, 64
    A, B = _adapters(wrng, C, d, d, rank, True)
    r = rng.integers(0, C, size=N).astype(np.int32)
    return Workload(name=f"f9-{N}", N=N, C=C, dtype="bf16", router="given", inputs={"x": _normal(rng, (N, d), 1.0, True)},
                    projections=[Projection("proj", "x", d, d, rank, A, B, _normal(rng, (N, d), 1.0, True))], r=r,
                    seq_id=np.arange(N, dtype=np.int32))


def t9_skew(kind: str, n_tokens: int = 2048) -> Workload:
    """Adapter-load skew at the conditions of Table 9: 4 adapters with the given load split (uniform, 80/10/5/5,
    95/2/2/1), one projection 4096->4096, rank 64, bf16.  Segment sizes are exact (largest-remainder rounding),
    token order is shuffled."""
    wrng, rng = _rng(8, 0), _rng(8, 1)
    N, C, d, rank = n_tokens, 4, 4096, 64
    share = np.asarray(T9_SKEWS[kind])
    sizes = np.floor(share * N).astype(int)
    sizes[: N - sizes.sum()] += 1
    r = np.repeat(np.arange(C, dtype=np.int32), sizes)
    rng.shuffle(r)
    A, B = _adapters(wrng, C, d, d, rank, True)
    return Workload(name=f"t9-{kind}", N=N, C=C, dtype="bf16", router="given", inputs={"x": _normal(rng, (N, d), 1.0, True)},
                    projections=[Projection("proj", "x", d, d, rank, A, B, _normal(rng, (N, d), 1.0, True))], r=r,
                    seq_id=np.arange(N, dtype=np.int32))


# Table 6 conditions: how the modalities are arranged inside the sequences.  The paper names three arrangements and gives
# neither their proportions nor the batch; these are this build's choices: 8 sequences of 256 tokens (its batch-256 point
# has the same per-token latency), d = 4096, r = 64, 4 modalities over the 160k vocabulary of the multimodal workload.
T6_KINDS = {"text-heavy": (0.70, 0.10, 0.10, 0.10), "balanced": (0.25, 0.25, 0.25, 0.25), "separated": None}


def t6_distribution(kind: str, n_seqs: int = 8, seq_len: int = 256) -> Workload:
    """Modality arrangement of Table 6: "text-heavy" and "balanced" interleave runs (geometric length, mean 16) whose
    modality is drawn with the given shares; "separated" gives every sequence one modality (sequence s: s mod 4).
    Vocabulary-routed, one projection 4096->4096, rank 64, bf16."""
    wrng, rng = _rng(6, 0), _rng(6, 1 + list(T6_KINDS).index(kind))
    N, C, d, rank = n_seqs * seq_len, 4, 4096, 64
    share = T6_KINDS[kind]
    mod = np.empty(N, dtype=np.int32)
    for s in range(n_seqs):
        if share is None:
            mod[s * seq_len:(s + 1) * seq_len] = s % C
            continue
        pos = 0
        while pos < seq_len:
            run = int(rng.geometric(1.0 / 16))
            mod[s * seq_len + pos: s * seq_len + min(seq_len, pos + run)] = int(rng.choice(C, p=share))
            pos += run
    lo = C5_BREAKS[:-1][mod].astype(np.int64)
    hi = C5_BREAKS[1:][mod].astype(np.int64)
    ids = (lo + (rng.random(N) * (hi - lo)).astype(np.int64)).astype(np.int32)
    A, B = _adapters(wrng, C, d, d, rank, True)
    return Workload(name=f"t6-{kind}", N=N, C=C, dtype="bf16", router="vocab", inputs={"x": _normal(rng, (N, d), 1.0, True)},
                    projections=[Projection("proj", "x", d, d, rank, A, B, _normal(rng, (N, d), 1.0, True))], ids=ids,
                    breaks=C5_BREAKS.copy(), seq_id=np.repeat(np.arange(n_seqs, dtype=np.int32), seq_len),
                    notes={"modality": mod})


SWEEP_NAMES = tuple(f"f9-{n}" for n in F9_BATCHES) + tuple(f"t9-{k}" for k in T9_SKEWS) + tuple(f"t6-{k}" for k in T6_KINDS)


def get(name: str, **kw) -> Workload:
    table = {"c1": c1_tiny_vocab, "c2": c2_prefill_1p7b, "c3": c3_decode_1p7b, "c4": c4_prefill_8b,
             "c5": c5_multimodal}
    if name == "c5-iid":
        return c5_multimodal(iid=True, **kw)
    if name.startswith("f9-"):
        return f9_batch(int(name[3:]))
    if name.startswith("t9-"):
        return t9_skew(name[3:], **kw)
    if name.startswith("t6-"):
        return t6_distribution(name[3:], **kw)
    return table[name](**kw)

"""Pins for the CPU oracle: each test checks it against something other than itself -- a value the
paper prints, a closed form, a library routine on a special case, or exhaustive enumeration on
exactly-representable data -- chosen so that a dropped term, a wrong sign or index, or a transposed
operand fails at least one of them.  CPU only."""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2603_15965_b200 import workloads as W


def _read_golden(path):
    out = {}
    with open(path) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, *vals = line.split()
            out[key] = np.array([int(v) for v in vals], dtype=np.int64)
    return out


def _small(seed, N=37, C=3, d_in=24, d_out=40, rank=4, dtype="f32", **kw):
    return W.random_problem(seed, N, C, d_in, d_out, rank, dtype, **kw)


# ------------------------------------------------------------------ top-k weighted routing (Eq. 8)
def test_topk_softmax_and_weighted_apply_pins():
    rng = np.random.default_rng(21)
    N, C, d_in, d_out, rank = 40, 5, 12, 9, 3
    z = rng.standard_normal((N, C))
    # k = 1: the argmax with weight exactly 1 (the case the hot path serves)
    i1, w1 = oracle.topk_softmax(z, 1)
    assert np.array_equal(i1[0], np.argmax(z, axis=1)) and np.all(w1 == 1.0)
    # k = 2: the two largest in order, weights in closed form: w_top = sigmoid(z_top - z_second), sum 1
    i2, w2 = oracle.topk_softmax(z, 2)
    order = np.argsort(-z, axis=1, kind="stable")
    assert np.array_equal(i2[0], order[:, 0]) and np.array_equal(i2[1], order[:, 1])
    gap = z[np.arange(N), i2[0]] - z[np.arange(N), i2[1]]
    assert np.allclose(w2[0], 1.0 / (1.0 + np.exp(-gap)), rtol=1e-13) and np.allclose(w2.sum(axis=0), 1.0, rtol=1e-13)
    # k = C: the full softmax (library routine), permuted into descending order
    from scipy.special import softmax
    i5, w5 = oracle.topk_softmax(z, C)
    assert np.allclose(w5.T, np.take_along_axis(softmax(z, axis=1), i5.T.astype(np.int64), axis=1), rtol=1e-12)
    # ties: equal logits are taken lowest index first
    it, wt = oracle.topk_softmax(np.array([[1.0, 3.0, 3.0, 0.0]]), 2)
    assert it[:, 0].tolist() == [1, 2] and np.allclose(wt[:, 0], [0.5, 0.5])
    # weighted apply: against library matmul per token; k = 1 with weight 1 equals the per-token apply of Eq. 2
    x = rng.standard_normal((N, d_in)).astype(np.float32)
    y = rng.standard_normal((N, d_out)).astype(np.float32)
    A = rng.standard_normal((C, d_in, rank)).astype(np.float32)
    B = rng.standard_normal((C, rank, d_out)).astype(np.float32)
    h = oracle.apply_topk(x, y, A, B, i2, w2, scale=0.5)
    ref = y.astype(np.float64).copy()
    for i in range(N):
        for j in range(2):
            c = i2[j, i]
            ref[i] += 0.5 * w2[j, i] * (x[i].astype(np.float64) @ A[c].astype(np.float64) @ B[c].astype(np.float64))
    assert np.allclose(h, ref, rtol=1e-12, atol=1e-12)
    h1 = oracle.apply_topk(x, y, A, B, i1, w1)
    ref1, _ = oracle.apply(x, y, A, B, i1[0])
    assert np.allclose(h1, ref1, rtol=1e-13, atol=1e-13)
    # swapping the two slots (with their weights) changes nothing: the sum over the kept set is order-free up to rounding
    hs = oracle.apply_topk(x, y, A, B, i2[::-1], w2[::-1], scale=0.5)
    assert np.allclose(hs, h, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ the paper's router (Eq. 9): 2-layer MLP, GELU
def test_mlp_router_pins():
    from scipy.stats import norm
    rng = np.random.default_rng(9)
    d, H, C, N = 10, 6, 4, 50
    x = rng.standard_normal((N, d)).astype(np.float32)
    W1 = rng.standard_normal((d, H)).astype(np.float32)
    b1 = rng.standard_normal(H).astype(np.float32)
    W2 = rng.standard_normal((H, C)).astype(np.float32)
    b2 = rng.standard_normal(C).astype(np.float32)
    r, z, margin, h = oracle.route_mlp(x, W1, b1, W2, b2, return_hidden=True)
    # hidden layer: GELU(t) = t * Phi(t) with Phi from an independent routine (the normal CDF), t by library matmul
    t = x.astype(np.float64) @ W1.astype(np.float64) + b1
    assert np.allclose(h, t * norm.cdf(t), rtol=1e-12, atol=1e-14)
    # output layer, argmax with lowest index on ties, margin = top1 - top2
    zz = h @ W2.astype(np.float64) + b2
    assert np.allclose(z, zz, rtol=1e-12, atol=1e-13)
    assert np.array_equal(r, np.argmax(zz, axis=1))
    srt = np.sort(zz, axis=1)
    assert np.allclose(margin, srt[:, -1] - srt[:, -2], rtol=1e-12, atol=1e-13)
    # unit vectors read rows of W1 (catches a transposed first layer); W2 = identity exposes the hidden layer
    _, z1, _, h1 = oracle.route_mlp(np.eye(d, dtype=np.float32), W1, None, np.eye(H, dtype=np.float32), None,
                                    return_hidden=True)
    assert np.allclose(h1, W1 * norm.cdf(W1.astype(np.float64)), rtol=1e-12, atol=1e-14) and np.array_equal(z1, h1)
    # closed forms: GELU(0) = 0, and far in the positive tail GELU is the identity, so the MLP collapses to the
    # (already pinned) linear gate with G = W1 W2 and bias = b1 W2 + b2
    r0, z0, _ = oracle.route_mlp(np.zeros((3, d), np.float32), W1, None, W2, b2)
    assert np.allclose(z0, np.broadcast_to(b2.astype(np.float64), (3, C)))
    big = (np.abs(W1) + 1.0).astype(np.float32)
    xb = (np.abs(x) + 1.0).astype(np.float32)
    bb = np.full(H, 40.0, np.float32)                              # pre-activations >= 40: Phi(t) == 1 in fp64
    rb, zb, _ = oracle.route_mlp(xb, big, bb, W2, b2)
    G = (big.astype(np.float64) @ W2.astype(np.float64))
    lin = xb.astype(np.float64) @ G + (bb.astype(np.float64) @ W2.astype(np.float64) + b2)
    assert np.allclose(zb, lin, rtol=1e-12) and np.array_equal(rb, np.argmax(lin, axis=1))
    # ties go to the lowest index: two identical output columns
    W2t = W2.copy(); W2t[:, 3] = W2t[:, 1]
    b2t = b2.copy(); b2t[3] = b2t[1]
    rt, zt, mt = oracle.route_mlp(x, W1, b1, W2t, b2t)
    assert not np.any(rt == 3) and np.all(mt[(rt == 1)] == 0.0)


# ------------------------------------------------------------------ grouping (Section 3.3, Figure 2)
def test_group_matches_figure2_example(golden_dir):
    g = _read_golden(os.path.join(golden_dir, "fig2_grouping.txt"))
    counts, offsets, perm = oracle.group(g["r"], 3)
    assert counts.tolist() == g["counts"].tolist()
    assert offsets.tolist() == g["offsets"].tolist()
    assert perm.tolist() == g["perm"].tolist()


@pytest.mark.parametrize("seed", range(6))
def test_group_invariants_and_library_sort(seed):
    rng = np.random.default_rng(seed)
    N, C = int(rng.integers(1, 400)), int(rng.integers(1, 40))
    r = rng.integers(-1, C, size=N).astype(np.int32)
    counts, offsets, perm = oracle.group(r, C)
    # histogram identity h[k] = |{t : r(t) = k}| (Table 10) via a library routine
    assert counts.tolist() == np.bincount(r[r >= 0], minlength=C).tolist()
    assert offsets[0] == 0 and np.array_equal(np.diff(offsets), counts)
    routed = np.flatnonzero(r >= 0)
    assert offsets[C] == routed.size == perm.size
    assert np.array_equal(np.sort(perm), routed)                     # a permutation of the routed tokens
    assert np.all(np.diff(r[perm]) >= 0)                              # grouped by adapter
    # stable: equals a library stable sort of the routed tokens by adapter
    assert np.array_equal(perm, routed[np.argsort(r[routed], kind="stable")])


def test_group_empty_and_single_adapter():
    counts, offsets, perm = oracle.group(np.zeros(0, np.int32), 4)
    assert counts.tolist() == [0, 0, 0, 0] and offsets.tolist() == [0] * 5 and perm.size == 0
    counts, offsets, perm = oracle.group(np.full(9, 2, np.int32), 3)
    assert counts.tolist() == [0, 0, 9] and perm.tolist() == list(range(9))


# ------------------------------------------------------------------ vocabulary routing (Definition 3.1)
def test_route_vocab_is_upper_bound_minus_one():
    rng = np.random.default_rng(1)
    breaks = np.array([0, 17, 17, 200, 1000, 4096], dtype=np.int32)       # includes an empty range
    ids = rng.integers(0, 4096, size=5000).astype(np.int32)
    ids[:12] = [0, 16, 17, 18, 199, 200, 201, 999, 1000, 4095, 1, 4094]    # every boundary
    expect = np.searchsorted(breaks, ids, side="right") - 1
    assert np.array_equal(oracle.route_vocab(ids, breaks), expect)


def test_route_vocab_c1_rule_and_out_of_range():
    w = W.get("c1")
    r = oracle.route_vocab(w.ids, w.breaks)
    assert np.array_equal(r, (w.ids >= 1000).astype(np.int32))             # ids < 1000 -> 0, >= 1000 -> 1
    r = oracle.route_vocab(np.array([-5, 0, 1999, 2000, 2**31 - 1], np.int32), w.breaks)
    assert r.tolist() == [-1, 0, 1, -1, -1]


def test_composite_target_range(golden_dir):
    # Example 3.3: c = a*|M| + m enumerates |A|*|M| distinct targets.
    g = _read_golden(os.path.join(golden_dir, "thm36_work.txt"))
    a, m = np.meshgrid(np.arange(64), np.arange(4), indexing="ij")
    c = a * 4 + m
    assert np.unique(c).size == int(g["composite_targets"][0]) and c.min() == 0 and c.max() == 255


def test_composite_routing_pins():
    # Definition 3.2 / Algorithm 1: c = a * |M| + m.  Pins: adapter 0 reduces to vocabulary routing; the pair (a, m)
    # is recovered by divmod; every one of the |A| * |M| targets of Example 3.3 is hit exactly once by one token per
    # (a, m); an id outside every range or an adapter outside [0, |A|) is unrouted.
    breaks = np.array([0, 100, 250, 251, 1000], np.int32)            # four ranges, one of a single id
    rng = np.random.default_rng(5)
    ids = rng.integers(0, 1000, size=500).astype(np.int32)
    m = oracle.route_vocab(ids, breaks)
    assert np.array_equal(oracle.route_composite(ids, np.zeros_like(ids), breaks, 64), m)
    a = rng.integers(0, 64, size=500).astype(np.int32)
    c = oracle.route_composite(ids, a, breaks, 64)
    assert np.array_equal(c // 4, a) and np.array_equal(c % 4, m)
    one_id_per_range = np.array([0, 100, 250, 251], np.int32)
    aa, mm = np.meshgrid(np.arange(64, dtype=np.int32), np.arange(4), indexing="ij")
    c = oracle.route_composite(one_id_per_range[mm.ravel()], aa.ravel(), breaks, 64)
    assert np.array_equal(np.sort(c), np.arange(256))
    c = oracle.route_composite(np.array([5, 1000, 5, -1], np.int32), np.array([3, 3, 64, 0], np.int32), breaks, 64)
    assert c.tolist() == [12, -1, -1, -1]


# ------------------------------------------------------------------ linear gate, top-1 (Eq. 8, k = 1)
def test_gate_unit_vectors_read_rows_of_G():
    rng = np.random.default_rng(2)
    d, C = 12, 5
    G = rng.standard_normal((d, C)).astype(np.float32)
    x = np.eye(d, dtype=np.float32)
    r, z, margin = oracle.route_gate(x, G)
    assert np.array_equal(z, G.astype(np.float64))                         # x = e_k  =>  z = G[k, :], catches a transposed G
    assert np.array_equal(r, np.argmax(G, axis=1))
    srt = np.sort(G.astype(np.float64), axis=1)
    assert np.array_equal(margin, srt[:, -1] - srt[:, -2])


def test_gate_equals_library_matmul_and_softmax_argmax():
    rng = np.random.default_rng(3)
    N, d, C = 200, 64, 7
    x = rng.standard_normal((N, d)).astype(np.float32)
    G = rng.standard_normal((d, C)).astype(np.float32)
    bias = rng.standard_normal(C).astype(np.float32)
    r, z, _ = oracle.route_gate(x, G, bias)
    zl = x.astype(np.float64) @ G.astype(np.float64) + bias.astype(np.float64)
    np.testing.assert_allclose(z, zl, rtol=1e-12, atol=1e-12)
    e = np.exp(zl - zl.max(axis=1, keepdims=True))
    p = e / e.sum(axis=1, keepdims=True)                                    # softmax is monotone: same winner
    assert np.array_equal(r, np.argmax(p, axis=1))
    # top-1 then softmax over the single kept logit gives weight exactly 1
    assert np.all(np.exp(zl.max(axis=1) - zl.max(axis=1)) == 1.0)


def test_gate_ties_go_to_lowest_index_and_planted_winner():
    x = np.ones((3, 4), dtype=np.float32)
    G = np.zeros((4, 6), dtype=np.float32)
    G[:, 2] = 1.0
    G[:, 4] = 1.0                                                           # columns 2 and 4 tie
    r, _, margin = oracle.route_gate(x, G)
    assert r.tolist() == [2, 2, 2] and np.all(margin == 0.0)
    rng = np.random.default_rng(4)
    xs = np.abs(rng.standard_normal((50, 8))).astype(np.float32)
    Gp = (0.01 * rng.standard_normal((8, 5))).astype(np.float32)
    Gp[:, 3] = 1.0                                                          # planted dominant adapter
    assert np.all(oracle.route_gate(xs, Gp)[0] == 3)


# ------------------------------------------------------------------ apply (Eq. 1, Eq. 2)
@pytest.mark.parametrize("c", [0, 2])
def test_constant_routing_reduces_to_dense_lora(c):
    # r == c everywhere is per-sequence routing with one adapter (Eq. 1): a dense LoRA by library matmul.
    w = _small(10)
    p = w.projections[0]
    x = w.inputs["x"]
    h, products = oracle.apply(x, p.y, p.A, p.B, np.full(w.N, c, np.int32))
    dense = p.y.astype(np.float64) + (x.astype(np.float64) @ p.A[c].astype(np.float64)) @ p.B[c].astype(np.float64)
    np.testing.assert_allclose(h, dense, rtol=1e-12, atol=1e-13)
    assert products == w.N


def test_general_routing_equals_grouped_library_matmul():
    # Figure 2's physical view: gather each adapter's tokens, one dense product per group, scatter back.
    w = _small(11, N=101, C=5, unrouted_frac=0.1)
    p = w.projections[0]
    x = w.inputs["x"].astype(np.float64)
    h, products = oracle.apply(w.inputs["x"], p.y, p.A, p.B, w.r, scale=0.5)
    ref = p.y.astype(np.float64).copy()
    for c in range(w.C):
        rows = np.flatnonzero(w.r == c)
        ref[rows] += 0.5 * (x[rows] @ p.A[c].astype(np.float64)) @ p.B[c].astype(np.float64)
    np.testing.assert_allclose(h, ref, rtol=1e-12, atol=1e-13)
    assert products == int(np.count_nonzero(w.r >= 0))
    unrouted = np.flatnonzero(w.r < 0)
    assert unrouted.size and np.array_equal(h[unrouted], p.y[unrouted].astype(np.float64))


def test_selector_adapters_closed_form():
    # A_c = e_j e_k^T, B_c = e_k e_o^T  =>  h[i][o] = y[i][o] + x[i][j] and every other column is y.
    N, C, d_in, d_out, rank = 9, 3, 7, 11, 4
    rng = np.random.default_rng(5)
    x = rng.standard_normal((N, d_in)).astype(np.float32)
    y = rng.standard_normal((N, d_out)).astype(np.float32)
    A = np.zeros((C, d_in, rank), np.float32)
    B = np.zeros((C, rank, d_out), np.float32)
    sel = [(1, 3, 10), (6, 0, 2), (4, 2, 5)]                                 # (j, k, o) per adapter, all distinct
    for c, (j, k, o) in enumerate(sel):
        A[c, j, k] = 1.0
        B[c, k, o] = 1.0
    r = rng.integers(0, C, size=N).astype(np.int32)
    h, _ = oracle.apply(x, y, A, B, r)
    expect = y.astype(np.float64).copy()
    for i in range(N):
        j, k, o = sel[r[i]]
        expect[i, o] += float(x[i, j])
    assert np.array_equal(h, expect)


def test_zero_B_and_unrouted_leave_y_untouched():
    w = _small(12)
    p = w.projections[0]
    h, _ = oracle.apply(w.inputs["x"], p.y, p.A, np.zeros_like(p.B), w.r)
    assert np.array_equal(h, p.y.astype(np.float64))
    h, products = oracle.apply(w.inputs["x"], p.y, p.A, p.B, np.full(w.N, -1, np.int32))
    assert np.array_equal(h, p.y.astype(np.float64)) and products == 0


def test_linearity_in_B_and_scale():
    w = _small(13)
    p = w.projections[0]
    x = w.inputs["x"]
    y0 = np.zeros_like(p.y)                                                  # y = 0 isolates the delta exactly
    d1, _ = oracle.apply(x, y0, p.A, p.B, w.r)
    d2, _ = oracle.apply(x, y0, p.A, 2.0 * p.B, w.r)                         # doubling B is exact in binary
    assert np.array_equal(d2, 2.0 * d1)
    ds, _ = oracle.apply(x, y0, p.A, p.B, w.r, scale=2.0)                    # scale folds into B
    assert np.array_equal(ds, d2)
    h, _ = oracle.apply(x, p.y, p.A, p.B, w.r)
    np.testing.assert_allclose(h, p.y.astype(np.float64) + d1, rtol=1e-15, atol=0)


def test_permutation_equivariance_bitwise():
    # Eq. 2 is row-independent: permuting the tokens permutes the result rows, bit for bit.
    w = _small(14, N=64, C=4)
    p = w.projections[0]
    x = w.inputs["x"]
    h, _ = oracle.apply(x, p.y, p.A, p.B, w.r)
    pi = np.random.default_rng(6).permutation(w.N)
    hp, _ = oracle.apply(x[pi], p.y[pi], p.A, p.B, w.r[pi])
    assert np.array_equal(hp, h[pi])


def test_work_counter_and_kpass_equivalence_exhaustive():
    # Theorem 3.6: per-token = N products, per-sequence K passes = K*N, identical results, all C^N routings.
    N, C, d_in, d_out, rank = 5, 3, 6, 4, 2
    rng = np.random.default_rng(7)
    x = rng.integers(-3, 4, size=(N, d_in)).astype(np.float32)
    y = rng.integers(-3, 4, size=(N, d_out)).astype(np.float32)
    A = rng.integers(-2, 3, size=(C, d_in, rank)).astype(np.float32)
    B = rng.integers(-2, 3, size=(C, rank, d_out)).astype(np.float32)
    for r in itertools.product(range(C), repeat=N):
        r = np.array(r, np.int32)
        h, n_tok = oracle.apply(x, y, A, B, r)
        hk, n_seq = oracle.apply_perseq_kpass(x, y, A, B, r)
        assert n_tok == N and n_seq == C * N
        assert np.array_equal(h, hk)
        # integer data: every product and sum is exact, so plain integer arithmetic must agree exactly
        xi, yi, Ai, Bi = (a.astype(np.int64) for a in (x, y, A, B))
        expect = np.stack([yi[i] + (xi[i] @ Ai[r[i]]) @ Bi[r[i]] for i in range(N)])
        assert np.array_equal(h, expect.astype(np.float64))


def test_work_counts_at_paper_operating_point(golden_dir):
    g = _read_golden(os.path.join(golden_dir, "thm36_work.txt"))
    N, K = int(g["N"][0]), int(g["K"][0])
    w = W.random_problem(15, N, K, 8, 8, 2, "f32")
    p = w.projections[0]
    h, n_tok = oracle.apply(w.inputs["x"], p.y, p.A, p.B, w.r)
    hk, n_seq = oracle.apply_perseq_kpass(w.inputs["x"], p.y, p.A, p.B, w.r)
    assert n_tok == int(g["per_token_products"][0]) and n_seq == int(g["per_sequence_products"][0])
    assert np.array_equal(h, hk)


def test_apply_rows_subset_is_exact():
    w = _small(16, N=80)
    p = w.projections[0]
    h, _ = oracle.apply(w.inputs["x"], p.y, p.A, p.B, w.r)
    rows = np.array([3, 79, 0, 41])
    assert np.array_equal(oracle.apply_rows(w.inputs["x"], p.y, p.A, p.B, w.r, rows), h[rows])


def test_thread_count_does_not_change_results():
    # the oracle is parallel over tokens only, so the number of OpenMP threads must not change a single bit: run the
    # same seeded problem in two fresh processes with 1 and with 4 threads and compare digests of every output
    import subprocess
    import sys
    code = (
        "import hashlib, sys, numpy as np, oracle\n"
        "from paper_2603_15965_b200 import workloads as W\n"
        "w = W.random_problem(17, 203, 5, 96, 72, 8, 'bf16', unrouted_frac=0.1)\n"
        "p = w.projections[0]\n"
        "G = np.random.default_rng(3).standard_normal((96, 5)).astype(np.float32)\n"
        "h, n = oracle.apply(w.inputs['x'], p.y, p.A, p.B, w.r)\n"
        "hk, nk = oracle.apply_perseq_kpass(w.inputs['x'], p.y, p.A, p.B, w.r)\n"
        "r, z, m = oracle.route_gate(w.inputs['x'], G)\n"
        "d = hashlib.sha256()\n"
        "for a in (h, hk, r, z, m): d.update(np.ascontiguousarray(a).tobytes())\n"
        "print(oracle.num_threads(), n, nk, d.hexdigest())\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    outs = []
    for threads in ("1", "4"):
        env = dict(os.environ, OMP_NUM_THREADS=threads, PYTHONPATH=root)
        res = subprocess.run([sys.executable, "-c", code], env=env, cwd=root, capture_output=True, text=True, check=True)
        outs.append(res.stdout.split())
    assert outs[0][0] == "1" and outs[1][0] == "4"              # the two runs really used different thread counts
    assert outs[0][1:] == outs[1][1:]


# ------------------------------------------------------------------ workload generator sanity (inputs only)
def test_workload_shapes_and_bf16_representable():
    w = W.get("c2", n_tokens=64)
    assert w.inputs["x"].shape == (64, 2048) and w.G.shape == (2048, 4)
    W.bf16_bits(w.inputs["x"])                                               # raises if not representable
    assert np.array_equal(W.bf16_bits_to_f32(W.bf16_bits(w.inputs["x"])), w.inputs["x"])
    r = np.array([1.0, 1.00390625, 1.01171875, -3.0e-40], np.float32)        # RNE on ties, denormal passthrough
    assert W.round_to_bf16(r)[1] == np.float32(1.0) and W.round_to_bf16(r)[2] == np.float32(1.015625)
    w3 = W.get("c3")
    assert [p.d_out for p in w3.projections] == [2048, 1024, 1024, 2048, 6144, 6144, 2048]
    assert np.array_equal(W.segment_sizes_routing([2, 0, 3]), np.array([0, 2, 0, 2, 2], np.int32))

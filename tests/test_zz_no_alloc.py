"""The allocation-free gate entry point (collected last: a failure here cannot hide other tests).

molora_route_gate_noalloc serves callers that cannot allocate device memory where they route tokens
(for example code between the capture and the replay of a fixed-address serving graph, or a plug-in that
is handed tensors but no allocator): its scratch is a fixed 2 MiB array inside the library instead of a
caller workspace.  It must give exactly what molora_route_gate gives -- same routing indices, same logits
within the tolerance the gate tests use -- also on the second of two calls in a row, when the shared scratch
still holds the first call's (different) contents."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import paper_2603_15965_b200 as M
from paper_2603_15965_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _problem(seed, N, d, C):
    rng = np.random.default_rng(seed)
    x = W.round_to_bf16(rng.standard_normal((N, d), dtype=np.float32))
    G = (rng.standard_normal((d, C)) * d ** -0.5).astype(np.float32)
    xd = torch.from_numpy(W.bf16_bits(x)).cuda().view(torch.bfloat16)
    return xd, torch.from_numpy(G).cuda()


def _call_noalloc(lib, x, G, r, logits):
    N, d = x.shape
    return lib.molora_route_gate_noalloc(ctypes.c_void_p(x.data_ptr()), M.BF16, N, d, x.stride(0),
                                         ctypes.c_void_p(G.data_ptr()), None, G.shape[1], ctypes.c_void_p(r.data_ptr()),
                                         ctypes.c_void_p(logits.data_ptr()), None)


def test_noalloc_gate_matches_workspace_gate_twice_in_a_row():
    lib = M.load_library()
    # different gates back to back, all on the tensor-core paths that need scratch (bf16, C > 4): the first two stay
    # below 1024 tokens (mma.sync gate), the third is large enough for the tcgen05 gate, which reads the split weights
    # from the library's array through a tensor map
    for seed, (N, d, C) in enumerate([(700, 4096, 16), (333, 2048, 8), (1500, 4096, 16), (1500, 4096, 16)]):
        x, G = _problem(seed, N, d, C)
        assert M.molora_route_gate_workspace_bytes(M.BF16, d, C) > 0
        ref_logits = torch.empty(N, C, dtype=torch.float32, device="cuda")
        ref_r = M.molora_route_gate(x, G, logits_out=ref_logits)
        r = torch.full((N,), -7, dtype=torch.int32, device="cuda")
        logits = torch.zeros(N, C, dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        assert _call_noalloc(lib, x, G, r, logits) == 0
        torch.cuda.synchronize()
        np.testing.assert_allclose(logits.cpu().numpy(), ref_logits.cpu().numpy(), rtol=1e-4, atol=1e-4)
        assert torch.equal(r, ref_r)
        # and directly against the CPU oracle: logits to 1e-4, argmax bit-exact outside the 1e-3 margin
        r_ref, z_ref, margin = oracle.route_gate(W.bf16_bits_to_f32(x.view(torch.int16).cpu().numpy().view(np.uint16)),
                                                 G.cpu().numpy())
        np.testing.assert_allclose(logits.cpu().numpy().astype(np.float64), z_ref, rtol=1e-4, atol=1e-4)
        keep = margin >= 1e-3
        assert np.array_equal(r.cpu().numpy()[keep], r_ref[keep])


def test_noalloc_gate_refuses_gates_beyond_its_scratch_and_handles_scratch_free_cases():
    lib = M.load_library()
    # the largest gate with 32 adapters that fits the 2 MiB array is accepted ...
    assert M.molora_route_gate_workspace_bytes(M.BF16, 8704, 32) <= (2 << 20)
    x, G = _problem(11, 16, 8704, 32)
    r = torch.full((16,), -7, dtype=torch.int32, device="cuda")
    logits = torch.zeros(16, 32, dtype=torch.float32, device="cuda")
    assert _call_noalloc(lib, x, G, r, logits) == 0
    torch.cuda.synchronize()
    assert torch.equal(r, M.molora_route_gate(x, G))
    # ... and the next width up is refused before anything is enqueued (real tensors: nothing here may fault even if
    # the refusal were ever lost)
    assert M.molora_route_gate_workspace_bytes(M.BF16, 8712, 32) > (2 << 20)
    x, G = _problem(12, 16, 8712, 32)
    r = torch.full((16,), -7, dtype=torch.int32, device="cuda")
    assert lib.molora_route_gate_noalloc(ctypes.c_void_p(x.data_ptr()), M.BF16, 16, 8712, x.stride(0),
                                         ctypes.c_void_p(G.data_ptr()), None, 32, ctypes.c_void_p(r.data_ptr()), None,
                                         None) == 3
    torch.cuda.synchronize()
    assert bool((r == -7).all())
    # C <= 4 needs no scratch and goes through as well
    x, G = _problem(5, 130, 512, 4)
    ref = M.molora_route_gate(x, G)
    assert torch.equal(M.molora_route_gate_noalloc(x, G), ref)

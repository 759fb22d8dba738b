"""The C-ABI library builds for sm_100a, loads, and exports every symbol the header declares; host-side
argument validation returns error codes before anything is enqueued.  No GPU needed (no compute calls)."""
import ctypes

import pytest

import paper_2603_15965_b200 as M
from paper_2603_15965_b200.build import build_library


def test_library_builds_loads_and_exports_header_symbols():
    build_library()
    lib = M.load_library()
    names = M.exported_symbols()
    assert {"molora_route_vocab", "molora_route_composite", "molora_route_mlp", "molora_route_mlp_workspace_bytes", "molora_topk_softmax", "molora_apply_topk",
            "molora_apply_topk_workspace_bytes", "molora_route_gate", "molora_group", "molora_apply", "molora_apply_batched", "molora_group_apply_batched",
            "molora_group_workspace_bytes", "molora_apply_workspace_bytes", "molora_route_gate_workspace_bytes",
            "molora_version", "molora_launch_count", "molora_debug_set",
            "molora_status_string"} <= set(names)
    for name in names:
        assert hasattr(lib, name), f"header declares {name} but the library does not export it"
    assert "sm_100a" in M.molora_version()
    assert M.molora_status_string(0) == "ok" and "workspace" in M.molora_status_string(3)


def test_invalid_arguments_are_refused_before_any_launch():
    lib = M.load_library()
    fake = ctypes.c_void_p(0x1000)      # never dereferenced: validation fails first
    # negative N
    assert lib.molora_route_vocab(fake, -1, fake, 2, fake, None, None) == 1
    # null breaks
    assert lib.molora_route_vocab(fake, 4, None, 2, fake, None, None) == 1
    # too many ranges
    assert lib.molora_route_vocab(fake, 4, fake, 257, fake, None, None) == 2
    # compositional routing: more than 256 composite targets, null adapter indices
    assert lib.molora_route_composite(fake, fake, 4, fake, 4, 65, fake, None, None) == 2
    assert lib.molora_route_composite(fake, None, 4, fake, 4, 64, fake, None, None) == 1
    # MLP router: hidden width and adapter count limits, tensor-core path without its workspace
    assert lib.molora_route_mlp(fake, M.BF16, 4, 64, 64, fake, None, 129, fake, None, 4, fake, None, None, 0, None, None) == 2
    assert lib.molora_route_mlp(fake, M.BF16, 4, 64, 64, fake, None, 64, fake, None, 33, fake, None, None, 0, None, None) == 2
    assert lib.molora_route_mlp(fake, M.BF16, 4, 64, 64, None, None, 64, fake, None, 4, fake, None, None, 0, None, None) == 1
    assert M.molora_route_mlp_workspace_bytes(M.BF16, 2560, 128, 4) == 2560 * 3 * 128 * 2
    assert M.molora_route_mlp_workspace_bytes(M.F32, 2560, 128, 4) == 0
    assert lib.molora_route_mlp(fake, M.BF16, 128, 64, 64, fake, None, 64, fake, None, 4, fake, None, None, 0, None, None) == 3
    # gate: d not a multiple of 8, C too large, pitch too small
    assert lib.molora_route_gate(fake, M.BF16, 4, 12, 16, fake, None, 4, fake, None, None, 0, None, None) == 2
    assert lib.molora_route_gate(fake, M.BF16, 4, 16, 16, fake, None, 33, fake, None, None, 0, None, None) == 2
    assert lib.molora_route_gate(fake, M.BF16, 4, 16, 8, fake, None, 4, fake, None, None, 0, None, None) == 1
    # tensor-core gate (bf16, C > 4) without its workspace
    assert M.molora_route_gate_workspace_bytes(M.BF16, 4096, 16) > 0 and M.molora_route_gate_workspace_bytes(M.BF16, 2048, 4) == 0
    assert lib.molora_route_gate(fake, M.BF16, 4, 16, 16, fake, None, 16, fake, None, None, 0, None, None) == 3
    # group: C out of range, null outputs
    assert lib.molora_group(fake, 4, 0, fake, fake, fake, None, 0, None, None) == 1
    assert lib.molora_group(fake, 4, 300, fake, fake, fake, None, 0, None, None) == 2
    assert lib.molora_group(fake, 4, 2, None, fake, fake, None, 0, None, None) == 1
    # apply: unsupported rank, misaligned pointer, bad dtype, null weights
    ok = dict(ldx=64, ldy=64, dt=M.BF16, N=4, d_in=64, d_out=64, rank=16, C=2)

    def apply(**kw):
        a = dict(ok, **kw)
        return lib.molora_apply(a.get("x", fake), a["ldx"], a.get("y", fake), a["ldy"], a["dt"], a["N"], a["d_in"],
                                a["d_out"], a["rank"], a.get("A", fake), a.get("B", fake), a["C"], fake, fake, 1.0,
                                None, 0, None, None)

    assert apply(rank=12) == 2
    assert apply(d_in=60) == 2
    assert apply(dt=7) == 2
    assert apply(x=ctypes.c_void_p(0x1004)) == 1
    assert apply(A=None) == 1
    assert apply(ldy=32) == 1
    assert apply(N=-3) == 1


@pytest.fixture
def default_kernels():
    """The library's own kernel choices before and after the test (overrides are process-wide)."""
    for k in M.TUNING_NAMES:
        M.molora_debug_set(k, 0)
    yield
    for k in M.TUNING_NAMES:
        M.molora_debug_set(k, 0)


def test_apply_workspace_sizes_and_refusal_without_it(default_kernels):
    lib = M.load_library()
    fake = ctypes.c_void_p(0x1000)
    # Two kernels need scratch.  (1) The two-launch small-tile kernels: fp32 partial shrink results [slice][N][rank];
    # forced here so that their figure stands alone:
    M.molora_debug_set("small_path", 2)
    # 256 tokens, d_in 2048, rank 64 -> 4 slices of 512 columns -> 4 * 256 * 64 * 4 bytes
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 64) == 4 * 256 * 64 * 4
    assert M.molora_apply_workspace_bytes(256, 8, 6144, 2048, 64) == 12 * 256 * 64 * 4
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 16) == 2 * 256 * 16 * 4
    M.molora_debug_set("small_path", 0)
    # (2) The job-list kernel (decode-sized calls: at most 1024 tokens, ranks 16 / 32 / 64): control words + partials.
    M.molora_debug_set("small_path", 3)
    ctl = 256                                                           # control words (CTAs finished, launches so far)
    # rank 16, d_in 2048: a full x-group (4 members) gets 384-column chunks -> 6 chunks; 256 / 16 + 8 = 24 tiles at most;
    # 16 x 16 records of 8 bytes {value, tag} per (tile, chunk)
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 16) == ctl + 24 * 6 * 16 * 16 * 8
    assert M.molora_apply_workspace_bytes(1025, 8, 2048, 2048, 16) == 0                 # more tokens than the kernel takes
    M.molora_debug_set("small_path", 0)
    # by default the job-list kernel takes rank 16 between 257 and 1024 tokens (with at least four projections, which is
    # not known here); rank 64 runs on the two-launch kernels while the projection moves less than ~12 MB (x once, y
    # twice) or has fewer than 256 tokens, on the tcgen05 kernel (no scratch) above
    assert M.molora_apply_workspace_bytes(512, 8, 2048, 2048, 16) == ctl + (512 // 16 + 8) * 6 * 16 * 16 * 8
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 16) == 0
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 32) == 0
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 64) == 4 * 256 * 64 * 4
    assert M.molora_apply_workspace_bytes(512, 8, 2048, 2048, 64) > 0          # 6.3 MB
    assert M.molora_apply_workspace_bytes(1024, 8, 2048, 2048, 64) == 0        # 12.6 MB
    assert M.molora_apply_workspace_bytes(1024, 64, 2048, 2048, 64) > 0        # 16-row segments on average: small tiles
    # larger calls of ranks 16 and 32 (streaming or tcgen05 kernel), rank 64 from 1280 tokens in any case, rank 8
    # and fp32-only shapes need none
    assert M.molora_apply_workspace_bytes(4096, 4, 2048, 2048, 16) == 0
    assert M.molora_apply_workspace_bytes(2048, 4, 2048, 2048, 32) == 0
    assert M.molora_apply_workspace_bytes(2048, 4, 2048, 2048, 64) == 0
    assert M.molora_apply_workspace_bytes(256, 8, 2048, 2048, 8) == 0
    assert M.molora_apply_workspace_bytes(256, 8, 2040, 2048, 64) == 0
    # with more than 64 adapters the short segments of a large rank-64 call take the two-launch kernels
    assert M.molora_apply_workspace_bytes(4096, 128, 2048, 2048, 64) > 0
    assert M.molora_apply_workspace_bytes(4096, 128, 2048, 2048, 16) == 0
    # a call that needs scratch is refused without it before anything is enqueued
    before = M.molora_launch_count()
    st = lib.molora_apply(fake, 64, fake, 64, M.BF16, 4, 64, 64, 64, fake, fake, 2, fake, fake, 1.0, None, 0, None, None)
    assert st == 3 and M.molora_launch_count() == before


def _desc(d_in, d_out, rank):
    from paper_2603_15965_b200.binding import _ProjDescC
    return _ProjDescC(0x1000, d_in, 0x2000, d_out, 0x3000, 0x4000, d_in, d_out, rank, 1.0, None)


def test_group_apply_one_call_launch_count_and_refusals(default_kernels):
    """Host arithmetic only: when molora_group_apply_batched is one launch, and that it validates both halves."""
    from paper_2603_15965_b200.binding import _ProjDescC
    lib = M.load_library()

    def one_launch(shapes, N, dt=M.BF16, C=8):
        arr = (_ProjDescC * len(shapes))(*[_desc(*s) for s in shapes])
        return int(lib.molora_group_apply_is_one_launch(arr, len(shapes), dt, N, C))

    assert one_launch([(2048, 2048, 16)], 4096) == 1                    # c2's apply: streaming kernel
    layer = [(2048, 2048, 16)] * 4 + [(2048, 6144, 16)] * 2 + [(6144, 2048, 16)]
    assert one_launch(layer, 256) == 1                                  # a decode layer: streaming kernel
    assert one_launch(layer, 512) == 1 and one_launch(layer, 1024) == 1 # ... job-list kernel (also one launch)
    assert one_launch([(2048, 2048, 16)], 4097) == 0                    # more tokens than a CTA groups on its own
    assert one_launch([(2048, 2048, 32)], 2048) == 1 and one_launch([(2048, 2048, 32)], 512) == 1   # rank 32 streams too
    assert one_launch([(2048, 2048, 64)], 512) == 0                     # rank 64, one projection: two-launch kernels
    assert one_launch([(2048, 2048, 64)] * 3, 512) == 1                 # rank 64, a layer's projections: streaming kernel
    arr64 = (_ProjDescC * 1)(_desc(2048, 2048, 64))
    assert int(lib.molora_group_apply_skips_group_launch(arr64, 1, M.BF16, 512, 8)) == 1    # two-launch kernels group on chip
    M.molora_debug_set("small_path", 2)
    M.molora_debug_set("umma_min_tokens", 1000000)
    assert int(lib.molora_group_apply_skips_group_launch(arr64, 1, M.BF16, 1100, 8)) == 0   # more than 1024 tokens: they do not
    assert one_launch([(2048, 2048, 16)], 4096) == 0
    M.molora_debug_set("small_path", 0)
    M.molora_debug_set("umma_min_tokens", 0)
    # rank 64 on the tcgen05 kernel (from ~12 MB with 256 tokens, from 1280 tokens in any case): it groups on chip, one
    # launch, up to 4096 tokens and 64 adapters
    assert one_launch([(2048, 2048, 64)] * 3, 2048) == 1
    assert one_launch([(4096, 4096, 64)], 1024) == 1 and one_launch([(4096, 4096, 64)], 4096) == 1
    assert one_launch([(4096, 4096, 64)], 4097) == 0 and one_launch([(4096, 4096, 64)], 2048, C=128) == 0
    assert one_launch([(2048, 2048, 16), (2048, 2048, 32)], 2048) == 0  # two ranks: two apply launches
    assert one_launch([(2048, 2048, 16)] * 8, 4096) == 1                # 400 MB: tcgen05 kernel, grouping inside
    assert one_launch([(2048, 2048, 16)] * 8, 8192) == 0                # ... beyond 4096 tokens: grouping launch + apply
    assert one_launch([(2048, 2048, 16)], 4096, M.F32) == 0             # fp32 storage: CUDA-core kernel
    assert one_launch([(2048, 2040, 16)], 256) == 0                     # width not a multiple of 32: CUDA-core kernel
    # refusals before any launch: null outputs, too many adapters, no projections, unsupported rank
    fake = ctypes.c_void_p(0x1000)
    arr = (_ProjDescC * 1)(_desc(64, 64, 16))
    assert lib.molora_group_apply_batched(fake, 8, 4, None, fake, fake, arr, 1, M.BF16, None, 0, None, None) == 1
    assert lib.molora_group_apply_batched(fake, 8, 257, fake, fake, fake, arr, 1, M.BF16, None, 0, None, None) == 2
    assert lib.molora_group_apply_batched(fake, 8, 4, fake, fake, fake, arr, 0, M.BF16, None, 0, None, None) == 1
    bad = (_ProjDescC * 1)(_desc(64, 64, 12))
    assert lib.molora_group_apply_batched(fake, 8, 4, fake, fake, fake, bad, 1, M.BF16, None, 0, None, None) != 0


def test_mixed_call_without_workspace_is_refused_before_any_launch(default_kernels):
    """A batched call whose projections need different kernels, one of them the two-launch kernels' scratch: with
    ws = NULL (or too small, or misaligned) the call must be refused as a whole, with nothing enqueued for the others."""
    from paper_2603_15965_b200.binding import _ProjDescC
    lib = M.load_library()
    fake = ctypes.c_void_p(0x1000)
    shapes = [(256, 512, 16), (512, 128, 64), (128, 192, 8), (200, 264, 32)]      # job-list kernel per rank, CUDA cores
    arr = (_ProjDescC * len(shapes))(*[_desc(*s) for s in shapes])
    need = sum(M.molora_apply_workspace_bytes(300, 6, *s) for s in shapes)
    assert need > 0
    before = M.molora_launch_count()
    assert lib.molora_apply_batched(arr, len(shapes), M.BF16, 300, 6, fake, fake, None, 0, None, None) == 3
    assert lib.molora_apply_batched(arr, len(shapes), M.BF16, 300, 6, fake, fake, fake, 4096, None, None) == 3    # too small
    assert lib.molora_apply_batched(arr, len(shapes), M.BF16, 300, 6, fake, fake, ctypes.c_void_p(0x1008), need, None, None) == 3
    assert lib.molora_group_apply_batched(fake, 300, 6, fake, fake, fake, arr, len(shapes), M.BF16, None, 0, None, None) == 3
    # the one-rank call that groups inside the two-launch kernels checks its scratch first as well
    arr64 = (_ProjDescC * 1)(_desc(512, 128, 64))
    assert lib.molora_group_apply_batched(fake, 300, 6, fake, fake, fake, arr64, 1, M.BF16, None, 0, None, None) == 3
    assert M.molora_launch_count() == before

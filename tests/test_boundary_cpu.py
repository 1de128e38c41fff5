"""Host-side checks that need no GPU: the C-ABI library loads and exports what the header declares,
its integer bookkeeping and argument validation behave as documented, the input generators are
deterministic, and the multi-process sharding covers every (batch, head) pair exactly once."""
import ctypes
import os
import re

import numpy as np
import pytest

import paper_2607_11897_b200 as sfda
import workloads
from oracle import bookkeeping
from paper_2607_11897_b200 import build as cuda_build
from paper_2607_11897_b200 import dp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    cuda_build.build()
    return sfda.load()


def test_library_exports_every_declared_symbol(lib):
    header = open(os.path.join(ROOT, "include", "sfda.h")).read()
    names = re.findall(r"SFDA_API\s+[\w\s\*]+?\b(sfda_\w+)\s*\(", header)
    assert len(names) >= 10 and len(set(names)) == len(names)
    for name in names:
        assert hasattr(lib, name), "libsfda.so does not export %s" % name


def test_plan_matches_integer_bookkeeping(lib):
    for T in (1, 5, 63, 64, 65, 256, 257, 8192, 131072):
        for chunk in (16, 32, 64):
            assert sfda.sfda_plan(T, chunk) == bookkeeping.chunk_plan(T, chunk)
    with pytest.raises(sfda.SfdaError) as e:
        sfda.sfda_plan(0, 64)
    assert e.value.status == -2


def test_status_strings(lib):
    seen = {sfda.sfda_status_string(c) for c in range(0, -9, -1)}
    assert len(seen) == 9 and "ok" in seen
    assert sfda.sfda_status_string(-99) == "unknown status"


def test_workspace_bytes(lib):
    # status block + one counter per (batch, head) + one boundary state per (batch, head) for the time slices
    assert sfda.sfda_workspace_bytes(8, 8192, 32, 128, 128, 64, sfda.SFDA_BF16) == 256 + 1024 + 256 * 128 * 128 * 4
    assert sfda.sfda_workspace_bytes(1, 256, 2, 64, 64, 16, sfda.SFDA_F32) == 0
    assert sfda.sfda_workspace_bytes(1, 256, 2, 128, 128, 64, sfda.SFDA_F32) == 0
    assert sfda.sfda_workspace_bytes(0, 256, 2, 128, 128, 64, sfda.SFDA_BF16) == 0


def test_host_arena_gives_every_piece_of_the_batch_an_aligned_beta_region(lib):
    """sfda_forward_host cuts the batch into at most eight pieces; beta has four bytes per (token, head), so a
    piece's share of one contiguous device array would leave the 16-byte grid whenever per * T * H is not a
    multiple of four.  The arena therefore reserves one 256-byte-rounded beta region per piece (host arithmetic)."""
    r256 = lambda x: (x + 255) // 256 * 256
    for B, T, H in ((2, 5, 1), (3, 130, 3), (9, 67, 1), (8, 64, 2), (17, 33, 5)):
        n, eb, d, m = B * T * H, 2, 128, 64
        per = (B + 7) // 8
        pieces = (B + per - 1) // per
        want = 2 * r256(n * d * eb) + r256(n * d * eb) + 2 * r256(n * m * 4) + 2 * r256(n * d * eb) \
            + r256(B * H * d * d * 4) + pieces * r256(per * T * H * 4) \
            + pieces * r256(sfda.sfda_workspace_bytes(per, T, H, d, d, 64, sfda.SFDA_BF16))
        assert sfda.sfda_forward_host_arena_bytes(B, T, H, d, d, 64, sfda.SFDA_BF16, True, True, True) == want
        assert (per * T * H * 4) % 16 != 0 or (B, T, H) in ((8, 64, 2),)      # the cases above do leave the grid


def test_a_library_built_from_other_sources_is_recognised(lib, tmp_path, monkeypatch):
    """The build records a hash of its sources beside the library; a tree whose sources differ from it (a file added,
    changed, or put back to an earlier state) makes the library stale whatever the file times say, and loading the
    package then rebuilds it."""
    assert not cuda_build.is_stale()
    h = cuda_build.source_hash()
    assert h == open(cuda_build.LIB + ".srchash").read().strip()
    assert cuda_build.source_hash(["-DSOMETHING"]) != h
    extra = tmp_path / "extra.cuh"
    extra.write_text("// one more header\n")
    deps = cuda_build._deps()
    monkeypatch.setattr(cuda_build, "_deps", lambda: sorted(deps + [str(extra)]))
    assert cuda_build.source_hash() != h and cuda_build.is_stale()


def test_chunks_of_128_and_256_tokens_are_superchunks_of_64_token_tiles(lib):
    """Section 6 ("superchunks": chunk transfers compose exactly): a chunk of 128 or 256 tokens runs as two or four
    64-token tiles, so the plan is the caller's, the workspace and the launcher's partition are those of the tiles, and
    other sizes stay unsupported; the factor export composes chunks of 128 and 256 tokens out of their tiles and needs
    all four factor arrays for it (host logic only)."""
    vp, ci = ctypes.c_void_p, ctypes.c_int
    for chunk in (128, 256):
        assert sfda.sfda_plan(1000, chunk) == bookkeeping.chunk_plan(1000, chunk)
        assert sfda.sfda_workspace_bytes(8, 8192, 32, 128, 128, chunk, sfda.SFDA_BF16) == \
            sfda.sfda_workspace_bytes(8, 8192, 32, 128, 128, 64, sfda.SFDA_BF16) > 0
        assert sfda.sfda_forward_partition(8, 8192, 32, 128, 128, chunk, sfda.SFDA_BF16, 1 << 30, 148) == \
            sfda.sfda_forward_partition(8, 8192, 32, 128, 128, 64, sfda.SFDA_BF16, 1 << 30, 148)
        assert sfda.sfda_forward_two_level_workspace_bytes(1, 131072, 16, 128, 128, chunk, sfda.SFDA_BF16, 0) == \
            sfda.sfda_forward_two_level_workspace_bytes(1, 131072, 16, 128, 128, 64, sfda.SFDA_BF16, 0) > 0
    assert sfda.sfda_workspace_bytes(1, 1024, 1, 128, 128, 512, sfda.SFDA_BF16) == 0
    assert sfda.sfda_workspace_bytes(1, 1024, 1, 128, 128, 96, sfda.SFDA_BF16) == 0
    ok = vp(0x1000)
    fac = lambda ptrs, d: lib.sfda_chunk_factors(*ptrs, *[ci(x) for x in d], None)
    assert fac([ok] * 4 + [ok] * 4 + [None], [1, 512, 1, 128, 512, 0]) == -3          # factors: up to 256 tokens
    assert fac([ok] * 4 + [ok, None, ok, ok] + [None], [1, 512, 1, 128, 256, 0]) == -1  # Y missing
    assert fac([ok] * 4 + [ok, ok, None, ok] + [None], [1, 256, 1, 128, 128, 0]) == -1  # M missing
    assert fac([ok] * 4 + [None, ok, ok, ok] + [None], [1, 256, 1, 128, 128, 0]) == -1  # Gamma missing
    # the diagnostic phase export is per 64-token tile
    ph = lambda chunk: lib.sfda_forward_phase(*([ok] * 6 + [None, ok, None, None]), ok,
                                              *[ci(d) for d in (1, 256, 1, 128, 128, chunk, 1)], vp(0x2000),
                                              ctypes.c_size_t(256), None)
    assert ph(128) == -3


def test_argument_validation_happens_before_any_launch(lib):
    """Every error below is found on the host; nothing touches a device (there is none here)."""
    vp, ci = ctypes.c_void_p, ctypes.c_int
    ok = vp(0x1000)                      # never dereferenced: validation fails first
    fwd = lambda ptrs, dims: lib.sfda_forward(*ptrs, *[ci(d) for d in dims], vp(0x2000), ctypes.c_size_t(256), None)
    base = [ok] * 6 + [None, ok, None, None]
    dims = [1, 64, 1, 128, 128, 64, 1]
    assert fwd([None] + base[1:], dims) == -1
    assert fwd(base, [0] + dims[1:]) == -2
    assert fwd(base, dims[:3] + [127] + dims[4:]) == -2          # odd d_k
    assert fwd(base, dims[:3] + [96] + dims[4:]) == -3
    assert fwd(base, dims[:5] + [48, 1]) == -3
    assert fwd(base, dims[:6] + [7]) == -3
    assert fwd([vp(0x1004)] + base[1:], dims) == -4
    assert lib.sfda_forward(*base, *[ci(d) for d in dims], None, ctypes.c_size_t(0), None) == -5
    step = lambda ptrs, d: lib.sfda_step(*ptrs, *[ci(x) for x in d], None)
    sbase = [ok] * 8 + [None]
    assert step([None] + sbase[1:], [1, 1, 128, 128, 1]) == -1
    assert step(sbase, [1, 0, 128, 128, 1]) == -2
    assert step(sbase, [1, 1, 128, 32, 1]) == -3
    fac = lambda ptrs, d: lib.sfda_chunk_factors(*ptrs, *[ci(x) for x in d], None)
    fbase = [ok] * 4 + [None] * 5
    assert fac([None] + fbase[1:], [1, 64, 1, 128, 64, 0]) == -1
    assert fac(fbase, [1, 64, 1, 128, 24, 0]) == -3
    n = lib.sfda_forward_host_arena_bytes(1, 64, 1, 128, 128, 64, 1, 1, 1, 1)
    assert n >= 64 * (3 * 256 + 2 * 256 + 4 + 2 * 256) + 65536
    assert lib.sfda_forward_host_arena_bytes(1, 64, 1, 100, 128, 64, 1, 1, 1, 1) == 0


def test_stable_parameterisation_entry_points_validate_on_the_host(lib):
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    ok = vp(0x1000)

    def front(ptrs, scal, dims):
        return lib.sfda_frontend(*ptrs[:4], *[cf(x) for x in scal], *ptrs[4:], *[ci(d) for d in dims], None)

    ptrs, scal, dims = [ok] * 8, [0.0, 1.0, 3.0, 1e-6], [1, 8, 1, 128, 1]

    def front_bwd(ptrs12, scal, dims):
        return lib.sfda_frontend_backward(*ptrs12[:4], *[cf(x) for x in scal], *ptrs12[4:], *[ci(d) for d in dims], None)

    lib.sfda_frontend_backward.restype = ci
    p12 = [ok] * 12                     # a, b, c, k_raw | dalpha, dtheta, dbeta, dk | da, db, dc, dk_raw
    assert front_bwd(p12[:7] + [None] + p12[8:], scal, dims) == -1          # dk
    assert front_bwd(p12[:11] + [None], scal, dims) == -1                     # dk_raw
    assert front_bwd(p12, scal, [1, 8, 1, 96, 1]) == -3
    assert front_bwd(p12[:4] + [vp(0x1004)] + p12[5:], scal, dims) == -4
    assert front_bwd(p12, [0.6, 0.5, 3.0, 0.0], dims) == -8
    assert front(ptrs[:3] + [None] + ptrs[4:], scal, dims) == -1
    assert front(ptrs, scal, [1, 0, 1, 128, 1]) == -2
    assert front(ptrs, scal, [1, 8, 1, 96, 1]) == -3
    assert front(ptrs, scal, [1, 8, 1, 128, 5]) == -3
    assert front([vp(0x1008)] + ptrs[1:], scal, dims) == -4
    for bad in ([-0.1, 1.0, 3.0, 0.0], [0.6, 0.5, 3.0, 0.0], [0.0, 1.5, 3.0, 0.0], [0.0, 1.0, -1.0, 0.0],
                [0.0, 1.0, 3.0, -1e-6], [float("nan"), 1.0, 3.0, 0.0], [0.0, 1.0, float("inf"), 0.0],
                [0.0, 1.0, 3.0, float("nan")]):
        assert front(ptrs, bad, dims) == -8, bad

    def fused(ptrs, scal, dims, ws=vp(0x2000), ws_bytes=1 << 30):
        return lib.sfda_forward_fused(*ptrs[:6], *[cf(x) for x in scal], *ptrs[6:], *[ci(d) for d in dims], ws,
                                      ctypes.c_size_t(ws_bytes), None)

    fptrs, fdims = [ok] * 6 + [None, ok, None, None], [1, 64, 1, 128, 128, 64, 1]
    assert fused([None] + fptrs[1:], scal, fdims) == -1
    assert fused(fptrs, scal, [1, 64, 0, 128, 128, 64, 1]) == -2
    assert fused(fptrs, scal, [1, 64, 1, 128, 96, 64, 1]) == -3
    assert fused(fptrs, [0.0, 2.0, 3.0, 0.0], fdims) == -8
    assert fused(fptrs, scal, fdims, ws=None, ws_bytes=0) == -5
    assert fused(fptrs, scal, [1, 64, 1, 64, 64, 16, 0], ws_bytes=1024) == -5      # staging does not fit
    def stepf(ptrs, scal, dims):
        return lib.sfda_step_fused(*ptrs[:6], *[cf(x) for x in scal], *ptrs[6:], *[ci(d) for d in dims], None)

    sptrs, sdims = [ok] * 8 + [None], [1, 1, 128, 128, 1]
    assert stepf([None] + sptrs[1:], scal, sdims) == -1
    assert stepf(sptrs, scal, [0, 1, 128, 128, 1]) == -2
    assert stepf(sptrs, scal, [1, 1, 128, 32, 1]) == -3
    assert stepf(sptrs, [0.0, 1.0, float("nan"), 0.0], sdims) == -8
    assert stepf(sptrs[:1] + [vp(0x1002)] + sptrs[2:], scal, sdims) == -4
    def stepd(ptrs, dims):
        return lib.sfda_step_decoupled(*ptrs, *[ci(d) for d in dims], None)

    #        q   k   r   v   al  th  eta be  S   o   o_im
    dptrs = [ok, ok, ok, ok, ok, ok, ok, ok, ok, ok, None]
    assert stepd(dptrs[:2] + [None] + dptrs[3:], sdims) == -1
    assert stepd(dptrs[:6] + [None] + dptrs[7:], sdims) == -1
    assert stepd(dptrs, [1, 0, 128, 128, 1]) == -2
    assert stepd(dptrs, [1, 1, 128, 48, 1]) == -3
    assert stepd(dptrs[:2] + [vp(0x1002)] + dptrs[3:], sdims) == -4
    def fwdd(ptrs, dims):
        return lib.sfda_forward_decoupled(*ptrs, *[ci(d) for d in dims], None)

    #         q   k   r   v   al  th  eta be  S0    o   o_im  S_T
    fdptrs = [ok, ok, ok, ok, ok, ok, ok, ok, None, ok, None, None]
    fddims = [1, 10, 2, 128, 64, 0]
    assert fwdd(fdptrs[:2] + [None] + fdptrs[3:], fddims) == -1
    assert fwdd(fdptrs[:6] + [None] + fdptrs[7:], fddims) == -1
    assert fwdd(fdptrs, [1, 0, 2, 128, 64, 0]) == -2
    assert fwdd(fdptrs, [1, 10, 2, 100, 64, 0]) == -3
    assert fwdd(fdptrs[:9] + [vp(0x1004)] + fdptrs[10:], fddims) == -4
    # workspace sizes: the tensor-core shape needs what sfda_forward needs; other shapes stage alpha, theta,
    # beta and the normalised key (each rounded up to 256 bytes)
    assert sfda.sfda_forward_fused_workspace_bytes(8, 8192, 32, 128, 128, 64, 1) == \
        sfda.sfda_workspace_bytes(8, 8192, 32, 128, 128, 64, 1)
    rows = 2 * 70 * 3
    r256 = lambda x: (x + 255) // 256 * 256
    assert sfda.sfda_forward_fused_workspace_bytes(2, 70, 3, 64, 64, 16, 0) == \
        2 * r256(rows * 32 * 4) + r256(rows * 4) + r256(rows * 64 * 4)
    assert sfda.sfda_forward_fused_workspace_bytes(2, 70, 3, 64, 64, 16, 1) == \
        2 * r256(rows * 32 * 4) + r256(rows * 4) + r256(rows * 64 * 2)
    assert sfda.sfda_forward_fused_workspace_bytes(2, 70, 3, 60, 64, 16, 1) == 0


def test_two_level_entry_point_validates_on_the_host(lib):
    vp, ci = ctypes.c_void_p, ctypes.c_int
    ok = vp(0x1000)

    def two(ptrs, dims, n, ws=vp(0x2000), ws_bytes=1 << 40):
        return lib.sfda_forward_two_level(*ptrs, *[ci(d) for d in dims], ci(n), ws, ctypes.c_size_t(ws_bytes), None)

    ptrs, dims = [ok] * 6 + [None, ok, None, None], [1, 2048, 2, 128, 128, 64, 1]
    assert two([None] + ptrs[1:], dims, 2) == -1
    assert two(ptrs, [1, 0, 2, 128, 128, 64, 1], 2) == -2
    assert two(ptrs, dims, 1) == -2 and two(ptrs, dims, -3) == -2
    assert two(ptrs, [1, 2048, 2, 64, 64, 16, 0], 2) == -3            # not a tensor-core shape
    assert two(ptrs, dims, 3) == -3                                    # 2048 tokens do not split into 3 x k x 64
    assert two(ptrs, dims, 64) == -3                                   # half a chunk per slice
    need = sfda.sfda_forward_two_level_workspace_bytes(1, 2048, 2, 128, 128, 64, 1, 2)
    r256 = lambda x: (x + 255) // 256 * 256
    states, tokens = 1 * 2 * 2 * 128 * 128 * 4, 1 * 2048 * 2 * 128 * 2
    assert need == r256(sfda.sfda_workspace_bytes(2, 1024, 2, 128, 128, 64, 1)) + 5 * r256(states) + 3 * r256(tokens)
    assert two(ptrs, dims, 2, ws_bytes=need - 1) == -5
    assert sfda.sfda_forward_two_level_workspace_bytes(1, 2048, 2, 128, 128, 64, 1, 3) == 0
    assert sfda.sfda_forward_two_level_workspace_bytes(1, 2048, 2, 64, 64, 16, 0, 2) == 0


def test_backward_entry_point_validates_on_the_host(lib):
    vp, ci = ctypes.c_void_p, ctypes.c_int
    ok = vp(0x1000)

    def bwd(ptrs, dims, ws=vp(0x2000), ws_bytes=1 << 40):
        return lib.sfda_backward(*ptrs, *[ci(d) for d in dims], ws, ctypes.c_size_t(ws_bytes), None)

    #       q   k   v   al  th  be  S0    do  do_im dS_T  dq  dk  dv  dal dth dbe dS0
    ptrs = [ok, ok, ok, ok, ok, ok, None, ok, None, None, ok, ok, ok, ok, ok, ok, ok]
    dims = [1, 100, 2, 128, 128, 1]
    assert bwd([None] + ptrs[1:], dims) == -1
    assert bwd(ptrs[:16] + [None], dims) == -1                       # every gradient is required
    assert bwd(ptrs, [1, 0, 2, 128, 128, 1]) == -2
    assert bwd(ptrs, [1, 100, 2, 96, 128, 1]) == -3
    assert bwd(ptrs, [1, 100, 2, 128, 128, 3]) == -3
    assert bwd(ptrs[:7] + [vp(0x1004)] + ptrs[8:], dims) == -4
    need = sfda.sfda_backward_workspace_bytes(1, 100, 2, 128, 128, 1)
    # 2 checkpoints + 64 states per (batch, head); two sequences split the columns into 4 blocks of 32, each with
    # its shares of dq, dk (128 each), dalpha, dtheta (64 each) and dbeta of the 200 (token, head) rows
    assert need == (1 * 2 * (2 + 64) * 128 * 128 + 4 * 200 * (3 * 128 + 1)) * 4
    # many sequences: one block, no shares
    assert sfda.sfda_backward_workspace_bytes(8, 128, 32, 128, 128, 1) == 8 * 32 * (2 + 64) * 128 * 128 * 4
    assert bwd(ptrs, dims, ws_bytes=need - 1) == -5
    assert bwd(ptrs, dims, ws=None, ws_bytes=0) == -5
    assert sfda.sfda_backward_workspace_bytes(1, 100, 2, 100, 128, 1) == 0


def test_block_control_entry_points_validate_on_the_host(lib):
    """sfda_forward_blocks / sfda_step_blocks: NULL, erase selector and alignment are refused before any launch."""
    import ctypes
    vp, ci = ctypes.c_void_p, ctypes.c_int
    fake = [vp(0x1000 + 0x100 * i) for i in range(13)]           # q k r v alpha theta flip eta beta S0 o o_im S_T
    lib.sfda_forward_blocks.restype = ci
    lib.sfda_step_blocks.restype = ci

    def fwd(ptrs, erase=0, dims=(1, 8, 2, 128, 128, 1)):
        return lib.sfda_forward_blocks(*ptrs, *[ci(x) for x in dims], ci(erase), None)

    assert fwd(fake[:2] + [None] + fake[3:]) == -1               # r
    assert fwd(fake[:7] + [None] + fake[8:]) == -1               # eta
    assert fwd(fake, erase=2) == -8
    assert fwd(fake[:6] + [vp(0x1004)] + fake[7:]) == -4         # flip
    assert fwd(fake, dims=(1, 8, 2, 96, 128, 1)) == -3
    step = [vp(0x1000 + 0x100 * i) for i in range(12)]           # q k r v alpha theta flip eta beta S o o_im

    def stp(ptrs, erase=0):
        return lib.sfda_step_blocks(*ptrs, ci(1), ci(2), ci(128), ci(128), ci(1), ci(erase), None)

    assert stp(step[:2] + [None] + step[3:]) == -1
    assert stp(step, erase=-1) == -8
    assert stp(step[:6] + [vp(0x1001)] + step[7:]) == -4
    assert stp(step[:9] + [None] + step[10:]) == -1              # S


def test_raw_input_generator_is_deterministic_and_untransformed():
    cfg = workloads.CONFIGS[1].scaled(B=2, T=64, H=2, s0_std=0.02)
    a, b = workloads.forward_raw_inputs(cfg), workloads.forward_raw_inputs(cfg)
    for key in a:
        assert np.array_equal(a[key], b[key])
    assert np.array_equal(workloads.forward_raw_inputs(cfg, batch=[1])["k_raw"][0], a["k_raw"][1])
    for key in ("q", "k_raw", "v"):
        assert np.array_equal(workloads.bf16_round(a[key]), a[key])
    n = np.linalg.norm(a["k_raw"].astype(np.float64), axis=-1)
    assert n.min() > 1.0 and n.max() / n.min() > 3.0                 # unnormalised, of varying length
    assert abs(a["a_raw"].mean() - 3.0) < 0.1 and a["b_raw"].std() > 1.3 and (a["c_raw"] < 0).any()


def test_missing_library_fails_loudly(monkeypatch):
    from paper_2607_11897_b200 import binding
    monkeypatch.setattr(binding, "_LIB", None)
    monkeypatch.setattr(binding, "lib_path", lambda: "/nonexistent/libsfda.so")
    with pytest.raises(ImportError):
        binding.load()


def test_generators_are_deterministic_and_on_the_storage_grid():
    cfg = workloads.CONFIGS[1].scaled(B=2, T=64, H=2, s0_std=0.02)
    a, b = workloads.forward_inputs(cfg), workloads.forward_inputs(cfg)
    for key in a:
        assert np.array_equal(a[key], b[key])
    one = workloads.forward_inputs(cfg, batch=[1])
    assert np.array_equal(one["q"][0], a["q"][1])                    # per-batch-element streams
    for key in ("q", "k", "v"):
        assert np.array_equal(workloads.bf16_round(a[key]), a[key])  # exactly representable in bf16
    assert np.abs(np.linalg.norm(a["k"].astype(np.float64), axis=-1) - 1).max() < 4e-3
    assert ((a["alpha"] > 0) & (a["alpha"] < 1)).all() and ((a["beta"] > 0) & (a["beta"] < 1)).all()
    # bf16 rounding: ties to even
    x = np.array([1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -9], np.float32)
    assert np.array_equal(workloads.bf16_round(x), np.array([1.0, 1.0 + 2 ** -6, 1.0], np.float32))
    c3 = workloads.CONFIGS[3].scaled(T=256, H=4)
    z = workloads.forward_batch_element(c3, 0)
    p = workloads.moduli(c3)
    j = np.rint(np.mod(z["theta"].astype(np.float64), 2 * np.pi) * p / (2 * np.pi))
    assert np.abs(np.mod(z["theta"].astype(np.float64), 2 * np.pi) - 2 * np.pi * j / p).max() < 1e-6
    assert set(np.unique(z["beta"])) <= {0.0, 1.0}


def _dp_worker(rank, world, port, out_dir):
    import torch
    import torch.distributed as dist
    from oracle import recurrence
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg = workloads.CONFIGS[0].scaled(B=3, T=32, H=2, s0_std=0.1)
    mine = list(dp.split_batch(cfg.B, world, rank))
    inp = workloads.forward_inputs(cfg, batch=mine)
    pairs = [(i, h) for i in range(len(mine)) for h in range(cfg.H)]
    s = workloads.sequences(inp, pairs)
    o_re, _, _ = recurrence.sfda_recurrence(s["q"], s["k"], s["v"], s["alpha"], s["theta"], s["beta"], s["S0"])
    np.save(os.path.join(out_dir, "o_%d.npy" % rank), o_re)
    np.save(os.path.join(out_dir, "b_%d.npy" % rank), np.array(mine))
    slowest = dp.max_over_ranks(1.0 + rank)            # rank r pretends to need 1 + r seconds
    assert slowest == float(world)
    assert dp.whole_job_throughput(10, world, slowest) == 10 * world / world
    dist.barrier()
    dist.destroy_process_group()


def test_two_process_sharding_needs_no_collective(tmp_path):
    import socket
    import torch.multiprocessing as mp
    from oracle import recurrence
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    world = 2
    mp.spawn(_dp_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    cfg = workloads.CONFIGS[0].scaled(B=3, T=32, H=2, s0_std=0.1)
    owned = np.concatenate([np.load(tmp_path / ("b_%d.npy" % r)) for r in range(world)])
    assert sorted(owned.tolist()) == list(range(cfg.B))           # every batch element exactly once
    inp = workloads.forward_inputs(cfg)
    pairs = [(b, h) for b in range(cfg.B) for h in range(cfg.H)]
    s = workloads.sequences(inp, pairs)
    want, _, _ = recurrence.sfda_recurrence(s["q"], s["k"], s["v"], s["alpha"], s["theta"], s["beta"], s["S0"])
    got = np.concatenate([np.load(tmp_path / ("o_%d.npy" % r)) for r in range(world)])
    assert np.array_equal(got, want)                              # shards simply concatenate
    assert list(dp.rank_batch_range(8, 3)) == list(range(24, 32))
    assert [len(dp.split_batch(7, 3, r)) for r in range(3)] == [3, 2, 2]


def test_forward_partition_rules():
    """How the forward spreads sequences over the SMs (host arithmetic of the launcher): time slices only when they
    shorten the schedule, none with fewer sequences than SMs (a sequence's slices run one after another), the
    balanced ranges only for shapes the slices cannot even out, nothing cut without the full workspace."""
    full = lambda B, H: sfda.sfda_workspace_bytes(B, 8192, H, 128, 128, 64, 1)
    part = lambda B, T, H, ws, sm=148: sfda.sfda_forward_partition(B, T, H, 128, 128, 64, 1, ws, sm)
    assert part(8, 8192, 32, full(8, 32)) == (4, 0, 148)          # headline: 1024 units, 7 rounds of 32 chunks
    assert part(8, 8192, 32, 256) == (1, 0, 148)                  # status block only: whole sequences
    assert part(4, 16384, 32, full(4, 32)) == (1, 0, 128)         # 128 sequences < 148 SMs: slicing buys nothing
    assert part(1, 131072, 16, full(1, 16)) == (1, 0, 16)
    assert part(16, 575, 19, full(16, 19)) == (1, 1, 148)         # 304 sequences of 9 chunks: balanced ranges
    assert part(4, 4113, 50, full(4, 50)) == (1, 1, 148)          # 200 sequences of 65 chunks
    assert part(5, 512, 40, full(5, 40)) == (2, 0, 148)           # 200 sequences of 8 chunks: two slices suffice
    assert part(8, 8192, 32, full(8, 32), sm=64) == (1, 0, 64)    # 256 sequences on 64 SMs: four even rounds
    assert sfda.sfda_forward_partition(1, 256, 2, 64, 64, 16, 0, 1 << 20, 148) == (1, 0, 0)   # CUDA-core path
    with pytest.raises(sfda.SfdaError):
        part(0, 64, 1, 256)


def test_balanced_ranges_cover_every_chunk_once():
    """The contiguous ranges the header defines for the balanced partition (CTA c starts at c*(N/ctas) +
    min(c, N % ctas)), walked the way the kernel walks them (last sequence of the range first): every chunk of
    every sequence exactly once, a sequence cut at most once, the head piece before anything else on its CTA and
    the tail piece last, so that no CTA waits for a piece that has not been started."""
    for B, T, H, sm in ((16, 575, 19, 148), (4, 4113, 50, 148), (1, 256, 149, 148), (3, 960, 60, 148), (1, 320, 101, 100)):
        slices, balanced, ctas = sfda.sfda_forward_partition(B, T, H, 128, 128, 64, 1,
                                                             sfda.sfda_workspace_bytes(B, T, H, 128, 128, 64, 1), sm)
        assert (slices, balanced, ctas) == (1, 1, sm)
        BH, NC = B * H, (T + 63) // 64
        N = BH * NC
        base, rem = divmod(N, ctas)
        seen, cuts = set(), {}
        for c in range(ctas):
            lo = c * base + min(c, rem)
            hi = lo + base + (1 if c < rem else 0)
            pieces = []
            bh = (hi - 1) // NC
            while bh * NC + NC > lo and bh >= 0:
                j0, j1 = max(lo - bh * NC, 0), min(hi - bh * NC, NC)
                pieces.append((bh, j0, j1))
                bh -= 1
            for n, (s, j0, j1) in enumerate(pieces):
                assert j0 < j1
                for j in range(j0, j1):
                    assert (s, j) not in seen
                    seen.add((s, j))
                if j1 < NC:                    # a head piece: first on its CTA
                    assert n == 0 and j0 == 0
                    cuts[s] = cuts.get(s, 0) + 1
                if j0 > 0:                     # a tail piece: last on its CTA
                    assert n == len(pieces) - 1 and j1 == NC
        assert len(seen) == N and all(v == 1 for v in cuts.values())

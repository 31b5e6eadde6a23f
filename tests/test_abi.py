"""The C-ABI library loads and exports every symbol include/cubicquant.h declares; host-side
size functions and argument validation (no compute, no GPU)."""
import ctypes
import os
import re

import pytest

import paper_2608_06763_b200 as cq

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cubicquant.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(cq_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = cq.lib()
    names = declared_functions()
    assert len(names) >= 16
    for n in names:
        assert hasattr(L, n), n


def test_sizes():
    assert cq.cq_canonical_code_bytes(4, 4096, 4096) == 4096 * 2048
    assert cq.cq_canonical_code_bytes(3, 2, 40) == 2 * 15
    # device layout has exactly the canonical byte count when N and K are multiples of 128
    for B in range(1, 9):
        for G in (32, 64, 128):
            assert cq.cq_layout_bytes(B, G, 256, 384) == 256 * 384 * B // 8 + 256 * (384 // G) * 8
            assert cq.cq_effective_bits(B, G) == B + 64 / G
    assert cq.cq_layout_bytes(4, 128, 130, 128) == 2 * (128 * 128 // 2 + 128 * 8)  # N padded to 256
    assert cq.cq_layout_bytes(4, 48, 128, 96) == 0 and cq.cq_layout_bytes(4, 128, 128, 192) == 0
    # G = 512: the record of a group is repeated in each of its four 128-wide tiles
    assert cq.cq_layout_bytes(4, 512, 128, 1024) == 128 * 1024 // 2 + 8 * 128 * 8
    assert cq.cq_workspace_bytes(4, 128, 1, 4096, 4096, cq.CQ_MODEL_DTYPE) > 0
    assert cq.cq_workspace_bytes(4, 128, 1, 4096, 4096, cq.CQ_DYN_A8) > cq.cq_workspace_bytes(4, 128, 1, 4096, 4096, 0)
    assert cq.cq_workspace_bytes(4, 128, 1, 4096, 4096, 7) == 0


def test_argument_errors_are_found_before_any_launch():
    L = cq.lib()
    one = ctypes.c_void_p(16)  # non-null, aligned, never dereferenced: validation fails first
    odd = ctypes.c_void_p(24)
    assert L.cq_gemm(None, 4, 128, one, one, 1, 128, 128, 0, one, 1 << 20, None) == -1
    assert L.cq_gemm(one, 9, 128, one, one, 1, 128, 128, 0, one, 1 << 20, None) == -1
    assert L.cq_gemm(one, 4, 128, one, one, 0, 128, 128, 0, one, 1 << 20, None) == -1
    assert L.cq_gemm(one, 4, 128, one, one, 1, 128, 128, 5, one, 1 << 20, None) == -1
    assert L.cq_gemm(one, 4, 128, one, one, 1, 128, 192, 0, one, 1 << 20, None) == -2   # K % G != 0
    assert L.cq_gemm(one, 4, 96, one, one, 1, 128, 192, 0, one, 1 << 20, None) == -2    # G unsupported
    assert L.cq_gemm(one, 4, 128, odd, one, 1, 128, 128, 0, one, 1 << 20, None) == -3
    assert L.cq_gemm(one, 4, 128, one, one, 1, 128, 128, 0, one, 16, None) == -4        # workspace too small
    assert L.cq_repack(None, one, one, one, 4, 128, 128, 128, one, None) == -1
    assert L.cq_quantize_a8(one, 0, 128, one, one, None) == -1
    assert L.cq_debug_wait_timeout(None, 512, 1000, None) == -1
    assert L.cq_debug_wait_timeout(one, 512, 0, None) == -1               # limit outside 1 .. 2e9
    assert L.cq_debug_wait_timeout(one, 512, 3 * 10 ** 9, None) == -1
    assert L.cq_debug_wait_timeout(one, 64, 1000, None) == -1             # too small to hold the status word
    assert L.cq_debug_wait_timeout(odd, 512, 1000, None) == -3
    assert cq.cq_status_string(-4) == "CQ_ERR_WORKSPACE"


def test_gemm_plan_shares_the_last_round_only_when_it_pays():
    """Host logic of the model-dtype GEMM's schedule (148 SMs are assumed when no device can be asked)."""
    L = cq.lib()
    plan = (ctypes.c_int64 * 5)()

    def ask(B, G, M, N, K, mode=0):
        assert L.cq_debug_gemm_plan(B, G, M, N, K, mode, plan) == 0
        return list(plan)

    assert L.cq_debug_gemm_plan(4, 128, 16, 4096, 4096, 0, plan) == -1    # M <= 16 is the small-M kernel's
    assert L.cq_debug_gemm_plan(4, 128, 64, 4096, 4096, 0, None) == -1
    assert L.cq_debug_gemm_plan(4, 128, 64, 4096, 4096, 7, plan) == -1
    for (M, N, K) in [(1024, 28672, 4096), (1024, 4096, 14336), (4096, 8192, 28672), (40, 256, 8192), (33, 100, 4224),
                      (4096, 57344, 8192), (1024, 6144, 4096), (17, 128, 128), (300, 200, 1024), (32, 28672, 4096)]:
        bnt, whole, runs, shared, crossing = ask(4, 128, M, N, K)
        tiles = -(-N // 128) * -(-M // bnt)
        kt = -(-K // 128)
        assert bnt in (32, 64, 128, 256, 512) and whole + shared == tiles
        if runs:
            assert shared < runs and whole % 148 == 0            # whole rounds, then the runs
            assert shared * kt >= 4 * runs                       # at least four layout tiles per run
            assert runs <= 148 if crossing else runs % shared == 0   # one run per SM, or the same number per tile
        else:
            assert shared == 0 and not crossing
    assert ask(4, 128, 1024, 28672, 4096) == [512, 444, 32, 4, 0]     # three whole rounds, four tiles cut into eight runs each
    assert ask(4, 128, 4096, 57344, 8192)[2] == 0                     # 24 rounds and a bit: sharing would not pay
    assert ask(4, 128, 17, 128, 128)[2] == 0                          # one layout tile of K cannot be cut
    # Dynamic A8: 256-token tiles at G = 128; only the tiles of the last round are cut, into equal slices
    assert ask(4, 128, 1024, 6144, 4096, 1) == [256, 148, 132, 44, 0]
    assert ask(4, 128, 300, 200, 512, 1)[2] == 0                      # four blocks of K: nothing to cut
    bn, whole, runs, shared, crossing = ask(4, 128, 100, 200, 2048, 1)
    assert (bn, whole, shared, crossing) == (128, 0, 2, 0) and runs in (4, 6, 8)

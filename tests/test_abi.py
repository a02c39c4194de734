"""The C-ABI library loads without a GPU and exports every function include/atb.h declares."""
import ctypes
import os
import re

import paper_2511_16041_b200 as atb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "atb.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(atb_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    lib = atb.load_library()
    names = declared_functions()
    assert "atb_gemm" in names and "atb_quantize_bfp16" in names and "atb_select_tiling" in names
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(atb.EXPORTED_SYMBOLS) == names


def test_binding_has_the_same_names():
    for n in declared_functions():
        assert callable(getattr(atb, n)), n


def test_status_strings_and_sizes():
    assert atb.atb_status_string(0) == "ATB_OK"
    assert atb.atb_status_string(8) == "ATB_ERR_DEVICE_TIMEOUT"
    assert atb.atb_status_string(99) == "ATB_ERR_UNKNOWN"
    assert atb.atb_bfp16_mant_bytes(100, 72) == 7200
    assert atb.atb_bfp16_exp_bytes(100, 72) == 2 * 128 * 8
    assert atb.atb_bfp16_exp_bytes(8192, 8192) == 8192 * 8192 // 8
    assert atb.atb_bfp16_exp_bytes(0, 64) == 0


def test_tiling_supported_rules():
    ok = atb.atb_tiling_supported
    assert ok(64, 128, 64, 128) and ok(128, 256, 64, 256) and ok(256, 256, 64, 256) and ok(32, 256, 64, 256)
    assert not ok(256, 128, 64, 128)          # T_MA > T_MC
    assert not ok(64, 192, 64, 128)           # T_MC not 128 / 256 / 384
    assert ok(64, 384, 64, 128) and ok(128, 384, 64, 128) and ok(32, 384, 128, 64)   # rho = 6, 3, 12
    assert not ok(256, 384, 64, 128) and not ok(128, 384, 64, 256)   # T_MA must divide T_MC; 3 x 256 columns > TMEM
    assert not ok(64, 128, 32, 128)           # T_K
    assert not ok(64, 128, 64, 96)            # T_N
    assert ok(128, 256, 64, 512) and ok(32, 256, 64, 512) and not ok(128, 256, 128, 512)   # CTA-pair tilings
    assert not ok(256, 256, 64, 512)          # a CTA of the pair holds 128 rows: no taller slab exists
    # asymmetric buffering is what makes the deep K-step fit next to a 256-wide B tile: two B tiles of
    # 128 x 256 take 128 KB, and the symmetric 256-row slabs do not fit beside them
    assert not ok(256, 256, 128, 256)
    assert ok(128, 256, 128, 256) and ok(64, 256, 128, 256) and ok(32, 256, 128, 256)


def test_layout_helpers_roundtrip():
    import numpy as np
    rng = np.random.default_rng(0)
    for (M, K) in [(100, 72), (32, 64), (33, 128), (1, 8)]:
        e = rng.integers(0, 255, size=(M, K // 8)).astype(np.uint8)
        plane = atb.logical_to_exp_plane(e, M, K)
        assert plane.size == atb.atb_bfp16_exp_bytes(M, K)
        assert np.array_equal(atb.exp_plane_to_logical(plane, M, K), e)
        # documented address rule: ((p * M_pad) + m) * 8 + (kb % 8)
        m_pad = -(-M // 32) * 32
        for (m, kb) in [(0, 0), (M - 1, K // 8 - 1), (M // 2, (K // 8) // 2)]:
            assert plane[((kb // 8) * m_pad + m) * 8 + kb % 8] == e[m, kb]


def test_argument_validation_needs_no_gpu():
    lib = atb.load_library()
    assert lib.atb_quantize_bfp16(None, 8, 12, 12, None, None, None) == 2       # K % 8
    assert lib.atb_quantize_bfp16(None, 0, 64, 64, None, None, None) == 0       # empty: no-op
    assert lib.atb_gemm(128, 128, 64, 64, 128, 64, 128, None, None, None, 128, None, 128, None) == 1
    assert lib.atb_gemm(128, 128, 72, 64, 128, 64, 128, 16, 16, 16, 128, 16, 128, None) == 2       # K % 16
    assert lib.atb_gemm_bfp16_out(128, 128, 64, 64, 128, 64, 128, 16, 16, 16, 128, None, 16, None) == 1   # NULL
    assert lib.atb_gemm_bfp16_out(128, 136, 64, 64, 128, 64, 128, 16, 16, 16, 136, 16, 16, None) == 2     # N % 16
    assert lib.atb_gemm_bfp16_out(128, 128, 64, 32, 128, 64, 128, 16, 16, 16, 128, 16, 16, None) == 3     # tiling
    assert lib.atb_gemm_config(0, 128, 128, 64, 16, None, 64, 16, 16, 16, None, 128, None) == 3            # config
    assert lib.atb_gemm_config(1, 128, 128, 64, 16, None, 64, 16, None, 16, None, 128, None) == 1          # NULL plane
    assert lib.atb_gemm_config(2, 128, 128, 64, 16, 16, 64, 16, 16, 16, None, 128, None) == 1              # config 2 needs C_exp
    assert lib.atb_gemm_config(1, 128, 136, 64, 16, None, 64, 16, 16, 16, None, 136, None) == 2            # N % 16
    assert lib.atb_gemm_config(1, 128, 128, 64, 24, None, 64, 16, 16, 16, None, 128, None) == 4            # alignment
    assert atb.atb_last_error_message() != ""


def test_ring_plans_fit_the_budgets():
    """Every supported tiling gets rings that fit 227 KB of shared memory and 512 TMEM columns; the
    barrier layout (lcm of depth and group count, see test_ring_protocol.py) stays small."""
    import math
    n = 0
    for mc in (128, 256, 384):
        for tn in (64, 128, 256, 512):
            for tk in (64, 128):
                for ma in (32, 64, 128, 256):
                    if ma > mc or mc % ma or not atb.atb_tiling_supported(ma, mc, tk, tn):
                        continue
                    p = atb.atb_tiling_plan(ma, mc, tk, tn)
                    n += 1
                    pair = (mc, tk, tn) == (256, 64, 512)
                    slab = min(ma, 128) if pair else ma
                    spg = max(128 // slab, 1)
                    bundle = spg                       # slabs converted per barrier round trip
                    while bundle > 1 and p.n_raw_stages % (bundle * p.dequant_groups):
                        bundle //= 2
                    stages = p.n_a_groups * (spg // bundle) if slab <= 128 else p.n_a_groups // (slab // 128)
                    assert p.dequant_groups in (1, 2, 4)
                    assert p.n_raw_stages >= p.dequant_groups and p.n_raw_stages % bundle == 0, (ma, mc, tk, tn)
                    assert stages >= 2, (ma, mc, tk, tn)
                    assert math.lcm(p.n_raw_stages, p.dequant_groups * bundle) <= 32
                    assert math.lcm(stages, p.dequant_groups) <= 32
                    assert p.n_b_stages >= 2 and p.acc_buffers in (1, 2)
                    assert p.smem_bytes <= 232448 and p.tmem_columns <= 512
                    assert p.tmem_columns >= p.acc_buffers * (128 if pair else mc) // 128 * tn
    assert n >= 30


def test_splitk_rejects_a_partial_tile_row_beyond_32_bits():
    """The FP32 partial tiles are addressed by a 32-bit row coordinate split * roundup(M, T_MC) + row:
    shapes whose product leaves that range are refused before anything is launched (host check only;
    the pointers are never dereferenced)."""
    lib = atb.load_library()
    M = 1 << 30
    big = lambda splits, fn, *tail: fn(M, 8, 128, 128, 256, 64, 128, 16, 16, 16, 8, 16, 8, splits, *tail)
    assert big(2, lib.atb_gemm_splitk, 16, 0, None) == 2                       # 2 * 2^30 rows: BAD_SHAPE
    assert "2^31" in atb.atb_last_error_message()
    assert big(2, lib.atb_gemm_splitk_noalloc, None) == 2
    assert big(1, lib.atb_gemm_splitk, 16, 0, None) == 7                       # in range: only the workspace is short
    assert big(1, lib.atb_gemm_splitk_noalloc, None) == 7                      # ... or larger than the built-in array

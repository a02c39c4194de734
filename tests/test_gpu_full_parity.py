"""GPU parity at full size: every element of C against the FP64 oracle for the cube workloads, and
sampled rows of every shape of the 125-shape sweep.

Asymmetric tile buffering only changes buffer lifetimes (Section 3): for any tiling the result is the
plain product.  The cube workloads check that claim at the benchmark's own launch configuration with
no sampling - every row of C goes through the oracle's GEMM and its acceptance test
|C_gpu - C_ref| <= 2^-7 |C_ref| + 2^-12 sum_k |a_ik b_kj| - for the tiling the selection picks, the
symmetric T_MA = T_MC ablation and the asymmetric form next to it.  The sweep (M, N, K in
{1024 .. 16384}^3, the shapes the model's ranking is measured on) checks the selected tiling and the
rho = 1, 2, 4, 8 family on the first and last row of every 256-row tile plus 64 random rows.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import bf16_bits_to_dev, bf16_dev_to_bits, dev

pytestmark = pytest.mark.gpu

RHO_FAMILY = [(256, 256, 64, 256), (128, 256, 64, 256), (64, 256, 64, 256), (32, 256, 64, 256)]
MAX_RATIO = 0.75          # one RNE to bf16 sits near 0.4 of the bound


def _logical_exp_rows(plane_d, M, K, rows_d):
    """Rows `rows_d` of the device exponent plane [ceil(K/64)][roundup(M,32)][8] as [rows][K/8] (layout only)."""
    panels, m_pad = -(-K // 64), -(-M // 32) * 32
    e = plane_d.view(panels, m_pad, 8)[:, rows_d, :].permute(1, 0, 2).reshape(rows_d.numel(), panels * 8)
    return e[:, :K // 8].cpu().numpy()


@pytest.mark.parametrize("name", ["cfg2_4096", "cfg3_8192"])
def test_every_element_of_the_cube_workloads(name):
    c = inputs.CONFIGS[name]
    M, N, K = c["M"], c["N"], c["K"]
    A, Bb = inputs.make_config(name)
    mant_d, plane_d = atb.atb_quantize_bfp16(torch.from_numpy(A).to(dev()))
    mant_o, exp_o = oracle.quantize_bfp16(A)
    del A
    # the device quantiser's planes, all of them, bit for bit
    assert np.array_equal(mant_d.cpu().numpy(), mant_o)
    assert np.array_equal(atb.exp_plane_to_logical(plane_d.cpu().numpy(), M, K), exp_o)
    Bd = bf16_bits_to_dev(Bb)
    selected = tuple(atb.atb_select_tiling(M, N, K)[0])
    tilings = list(dict.fromkeys([selected, (256, 256, 64, 256), (128, 256, 64, 256)]))
    results = {}
    for t in tilings:
        C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
        atb.atb_gemm(M, N, K, *t, mant_d, plane_d, Bd, C)
        atb.atb_device_status()
        results[t] = bf16_dev_to_bits(C)
        del C
    # the symmetric and the asymmetric tiling add the same products in the same order
    assert np.array_equal(results[(256, 256, 64, 256)], results[(128, 256, 64, 256)])
    worst = {t: 0.0 for t in tilings}
    chunk = 1024                                     # C_ref and S of a chunk: 2 x 64 MB at N = 8192
    for r0 in range(0, M, chunk):
        rows = np.arange(r0, min(r0 + chunk, M), dtype=np.int64)
        Cr, S = oracle.gemm(mant_o, exp_o, Bb, rows=rows)
        for t in tilings:
            bad, ratio = oracle.check_tolerance(results[t][rows], Cr, S)
            assert bad == 0, (name, t, r0, bad, ratio)
            worst[t] = max(worst[t], ratio)
    for t in tilings:
        assert worst[t] < MAX_RATIO, (name, t, worst[t])


def _sweep_rows(M, seed):
    edges = np.concatenate([np.arange(0, M, 256), np.arange(255, M, 256)])
    rnd = np.random.default_rng(seed).integers(0, M, 64)
    return np.unique(np.concatenate([edges, rnd])).astype(np.int64)


@pytest.mark.parametrize("K", inputs.SWEEP_SIZES)
@pytest.mark.parametrize("N", inputs.SWEEP_SIZES)
def test_sweep_shapes_sampled_rows(N, K):
    """The five M of the sweep for one (N, K): operands drawn on the device, the sampled rows of A
    copied back so that the oracle quantises and multiplies exactly what the device was given."""
    Bd = inputs.device_normal((K, N), inputs.BASE_SEED, inputs.TAG_B, dev(), torch.bfloat16)
    Bb = bf16_dev_to_bits(Bd)
    for M in inputs.SWEEP_SIZES:
        Ad = inputs.device_normal((M, K), inputs.BASE_SEED + M, inputs.TAG_A, dev())
        mant_d, plane_d = atb.atb_quantize_bfp16(Ad)
        rows = _sweep_rows(M, M + N + K)
        rows_d = torch.from_numpy(rows).to(dev())
        mant_o, exp_o = oracle.quantize_bfp16(Ad[rows_d].cpu().numpy())
        del Ad
        assert np.array_equal(mant_d[rows_d].cpu().numpy(), mant_o), (M, N, K)
        assert np.array_equal(_logical_exp_rows(plane_d, M, K, rows_d), exp_o), (M, N, K)
        Cr, S = oracle.gemm(mant_o, exp_o, Bb)
        selected = tuple(atb.atb_select_tiling(M, N, K)[0])
        C = torch.empty((M, N), dtype=torch.bfloat16, device=dev())
        family = None
        for t in [selected] + RHO_FAMILY:
            C.fill_(float("nan"))
            atb.atb_gemm(M, N, K, *t, mant_d, plane_d, Bd, C)
            atb.atb_device_status()
            if t in RHO_FAMILY:                      # same (T_MC, T_K, T_N): bit-identical whatever rho is
                if family is None:
                    family = C.clone()
                else:
                    assert torch.equal(C.view(torch.int16), family.view(torch.int16)), (M, N, K, t)
                    continue
            bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(C[rows_d]), Cr, S)
            assert bad == 0 and ratio < MAX_RATIO, (M, N, K, t, bad, ratio)
            assert bool(torch.isfinite(C.float()).all()), (M, N, K, t)
        del C, family, mant_d, plane_d

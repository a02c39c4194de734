"""Randomised parity and run-to-run determinism of the GEMM kernels.

A data race between the kernel's roles (TMA producer, dequantisers, UMMA issuer, epilogue) would
show up as a run-to-run difference or as a tolerance failure on some shape; both are checked here.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2511_16041_b200 as atb
from paper_2511_16041_b200 import inputs
from tests.gpu_util import dev, planes_to_dev, bf16_bits_to_dev, bf16_dev_to_bits

pytestmark = pytest.mark.gpu


def _all_tilings():
    return [(ma, mc, k, n) for mc in (128, 256) for n in (64, 128, 256, 512) for k in (64, 128)
            for ma in (32, 64, 128, 256) if ma <= mc and atb.atb_tiling_supported(ma, mc, k, n)]


def test_random_shapes_and_tilings_against_oracle():
    rng = np.random.default_rng(20251116)
    tilings = _all_tilings()
    kinds = ["normal", "laplace", "outlier"]
    for case in range(40):
        M = int(rng.integers(1, 1400))
        N = int(rng.integers(1, 130)) * 8
        K = int(rng.integers(1, 100)) * 16
        t = tilings[int(rng.integers(0, len(tilings)))]
        A = inputs.make_A(kinds[case % 3], M, K, inputs.BASE_SEED + case)
        Bb = inputs.make_B_bits(K, N, 1.0, inputs.BASE_SEED + case)
        mant, exp = oracle.quantize_bfp16(A)
        md, ed = planes_to_dev(mant, exp)
        Bd = bf16_bits_to_dev(Bb)
        C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
        atb.atb_gemm(M, N, K, *t, md, ed, Bd, C)
        atb.atb_device_status()
        Cr, S = oracle.gemm(mant, exp, Bb)
        bad, ratio = oracle.check_tolerance(bf16_dev_to_bits(C), Cr, S)
        assert bad == 0 and ratio < 0.75, (case, (M, N, K), t, bad, ratio)


@pytest.mark.parametrize("tiling", [(128, 256, 64, 256), (64, 256, 64, 256), (32, 128, 64, 128), (128, 256, 64, 512),
                                     (64, 256, 128, 128)])
def test_run_to_run_bitwise_determinism(tiling):
    """Many tiles per CTA and many K-steps: ring phases wrap often; five runs must agree bit for bit."""
    M, N, K = 4096, 2048, 4096
    g = torch.Generator(device=dev())
    g.manual_seed(7)
    mant = torch.randint(-127, 128, (M, K), dtype=torch.int8, device=dev(), generator=g)
    plane = torch.randint(120, 135, (atb.atb_bfp16_exp_bytes(M, K),), dtype=torch.uint8, device=dev(), generator=g)
    B = torch.randn((K, N), device=dev(), generator=g).to(torch.bfloat16)
    ref = None
    for run in range(5):
        C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
        atb.atb_gemm(M, N, K, *tiling, mant, plane, B, C)
        atb.atb_device_status()
        assert bool(torch.isfinite(C.float()).all())
        if ref is None:
            ref = C.view(torch.int16).clone()
        assert torch.equal(C.view(torch.int16), ref), (tiling, run)
    # and a sampled comparison against the oracle on this large case
    rows = np.unique(np.random.default_rng(3).integers(0, M, 24)).astype(np.int64)
    mant_h = mant[torch.from_numpy(rows).to(dev())].cpu().numpy()
    exp_h = atb.exp_plane_to_logical(plane.cpu().numpy(), M, K)[rows]
    Cr, S = oracle.gemm(mant_h, exp_h, bf16_dev_to_bits(B))
    got = bf16_dev_to_bits(ref.view(torch.bfloat16)[torch.from_numpy(rows).to(dev())])
    bad, ratio = oracle.check_tolerance(got, Cr, S)
    assert bad == 0 and ratio < 0.75, (tiling, bad, ratio)


def test_calibration_measures_and_fits_on_this_gpu(tmp_path):
    """The calibration tool end to end on two small shapes and a handful of tilings."""
    from paper_2511_16041_b200 import calibrate
    tilings = [(128, 256, 64, 256), (64, 256, 64, 256), (128, 128, 64, 256), (128, 256, 64, 128), (128, 256, 64, 512)]
    records = calibrate.measure([(2048, 2048, 2048), (1024, 4096, 1024)], tilings, reps=3)
    assert len(records) == 10 and all(r["tflops"] > 10 for r in records)
    values, ev = calibrate.fit(records, {"convert_cycles": (300.0, 400.0), "load_latency_cycles": (1200.0, 2000.0)})
    assert set(values) == {"convert_cycles", "load_latency_cycles"} and 0.5 < ev["pick_quality_mean"] <= 1.0


def test_quantise_and_gemm_capture_into_a_cuda_graph():
    """The entry points only enqueue work on the given stream (tensor maps travel by value as kernel
    parameters), so a step can be captured once and replayed: the replay gives the eager result bit for
    bit, also after the input buffers were refilled."""
    device = dev()
    gen = torch.Generator(device=device)
    gen.manual_seed(5)
    M, N, K = 1000, 1544, 1104
    A = torch.randn((M, K), device=device, generator=gen)
    B = torch.randn((K, N), device=device, generator=gen).to(torch.bfloat16)
    mant = torch.empty((M, K), dtype=torch.int8, device=device)
    plane = torch.empty(atb.atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=device)
    eager = torch.empty((M, N), dtype=torch.bfloat16, device=device)
    replayed = torch.zeros((M, N), dtype=torch.bfloat16, device=device)
    s = torch.cuda.Stream(device)
    for tiling in [(128, 256, 64, 256), (128, 256, 64, 512)]:
        def step(out):
            atb.atb_quantize_bfp16(A, mant, plane, stream=s)
            atb.atb_gemm(M, N, K, *tiling, mant, plane, B, out, stream=s)
        with torch.cuda.stream(s):
            step(eager)                      # also the warm-up the capture needs
        s.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            step(replayed)
        for _ in range(2):
            replayed.zero_()
            graph.replay()
            torch.cuda.synchronize()
            with torch.cuda.stream(s):
                step(eager)
            s.synchronize()
            assert torch.equal(eager, replayed), tiling
            A.mul_(1.5)                      # new values in the same buffers for the second round
    atb.atb_device_status()


def test_soak_cta_pair_against_single_cta_bitwise():
    """A bounded soak of the CTA-pair kernel: its dequantisers announce an operand to the leader CTA with
    a CTA-scope release (the operand is read by the announcing CTA's own tensor core only), which the
    memory model does not promise to order against the leader's cluster-scope acquire.  Random shapes
    (ragged edges, one to hundreds of K-steps), the three slab heights of the pair and - where no CTA
    computes more than one tile, so that both kernels add the same products in the same order - the
    single-CTA 256 x 256 tiling: all results must be bit-identical, launch after launch.  The stacked pair
    (two 128 x 256 tiles on a pair) runs the same hand-over: its three slab heights must agree bit for bit
    with one another at every size, and with all the others where every kernel has one tile per CTA."""
    import random
    import time
    g = torch.Generator(device=dev())
    g.manual_seed(11)
    rnd = random.Random(5)
    pair_tilings = [(128, 256, 64, 512), (64, 256, 64, 512), (32, 256, 64, 512)]
    stacked_tilings = [(128, 128, 128, 256), (64, 128, 128, 256), (32, 128, 128, 256)]
    launches, t_end = 0, time.time() + 12.0
    while time.time() < t_end or launches < 400:
        M = rnd.choice([300, 1000, 2048, 4096, 5000])
        N = rnd.choice([512, 1024, 2048, 4104])
        K = rnd.choice([16, 64, 448, 1024, 1104, 4096])
        one_wave = -(-M // 256) * -(-N // 256) <= 148 and -(-M // 256) * -(-N // 512) <= 74
        tilings = ([(128, 256, 64, 256)] if one_wave else []) + pair_tilings
        stacked_one_wave = one_wave and -(-M // 256) * -(-N // 256) <= 74
        mant = torch.randint(-127, 128, (M, K), dtype=torch.int8, device=dev(), generator=g)
        plane = torch.randint(100, 150, (atb.atb_bfp16_exp_bytes(M, K),), dtype=torch.uint8, device=dev(), generator=g)
        B = torch.randn((K, N), device=dev(), generator=g).to(torch.bfloat16)
        ref = ref_stacked = None
        for rep in range(6):
            for t in tilings:
                C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
                atb.atb_gemm(M, N, K, *t, mant, plane, B, C)
                launches += 1
                if ref is None:
                    ref = C.view(torch.int16).clone()
                else:
                    assert torch.equal(C.view(torch.int16), ref), ((M, N, K), t, rep)
            if rep < 2:
                for t in stacked_tilings:
                    C = torch.full((M, N), float("nan"), dtype=torch.bfloat16, device=dev())
                    atb.atb_gemm(M, N, K, *t, mant, plane, B, C)
                    launches += 1
                    if ref_stacked is None:
                        ref_stacked = ref if stacked_one_wave else C.view(torch.int16).clone()
                    assert torch.equal(C.view(torch.int16), ref_stacked), ((M, N, K), t, rep)
        atb.atb_device_status()
        assert bool(torch.isfinite(ref.view(torch.bfloat16).float()).all())
    assert launches >= 400

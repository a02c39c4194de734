"""The library's host-side model (C++) against the oracle's restatement of Sections 3-5."""
import math
import os

import pytest

import paper_2511_16041_b200 as atb
from oracle import model
from tests.test_oracle_model import rows, _printed


@pytest.mark.parametrize("r", rows(), ids=lambda r: f"{r['cfg']}-{r['T_MC']}x{r['T_K']}x{r['T_N']}-rho{r['rho']}")
def test_xdna2_preset_reproduces_table2(r):
    cfg = int(r["cfg"][1])
    hw = atb.atb_hw_params_xdna2(cfg)
    T_MA = r["T_MC"] // r["rho"]
    s = atb.atb_score_tiling(hw, r["K"], (T_MA, r["T_MC"], r["T_K"], r["T_N"]))
    assert abs(s.ai - r["ai"]) <= 0.5
    assert abs(s.mem_bound_flops / 1e12 - r["mem"]) <= 0.075
    if r["buf"] != "-":
        assert _printed(s.buf_bytes_used / 1024, r["buf"])
        assert s.feasible == 1
        if r["rho"] > 1:
            sym = atb.atb_score_tiling(hw, r["K"], (r["T_MC"], r["T_MC"], r["T_K"], r["T_N"]))
            assert sym.feasible == 0


def test_score_matches_oracle_formulas():
    for hw in (atb.atb_hw_params_b200(), atb.atb_hw_params_xdna2(1), atb.atb_hw_params_xdna2(3)):
        for t in [(32, 256, 64, 256), (128, 128, 128, 64), (64, 256, 128, 128), (256, 256, 64, 256)]:
            for K in (256, 4096, 16384):
                s = atb.atb_score_tiling(hw, K, t)
                T_MA, T_MC, T_K, T_N = t
                ai = model.ai_array(T_MC, T_N, K, hw.a_bytes, hw.b_bytes, hw.c_bytes, hw.share_rows, hw.share_cols)
                em = model.eff_micro(T_K, hw.eta, hw.eps_cycles, hw.ii)
                # rho_eff of the preset: a slab larger than the MMA's M extent is consumed in pieces; a thinner
                # one is bundled and costs thin_slab_cost of a switch beyond the first of its bundle
                rho_eff = T_MC / T_MA
                if hw.mma_rows > 0:
                    per_mma = T_MC / hw.mma_rows
                    if T_MA > hw.mma_rows:
                        rho_eff = per_mma
                    elif T_MA < hw.mma_rows:
                        rho_eff = per_mma + (T_MC / T_MA - per_mma) * hw.thin_slab_cost
                ec = model.eff_core(T_MC / rho_eff, T_MC, T_K, T_N, hw.peak_flops_per_cycle, em, hw.delta_cycles)
                if hw.mma_rows > 0 and T_MA > hw.mma_rows and hw.coarse_slab_factor > 0:
                    ec *= hw.coarse_slab_factor
                if hw.mma_rows > 0 and T_K > 64 and hw.deep_kstep_factor > 0:
                    ec *= hw.deep_kstep_factor
                if hw.mma_rows > 0 and (hw.convert_cycles > 0 or hw.convert_exposed_cycles > 0):
                    # conversion of A on the compute side: a unit of mma_rows x 64 elements feeds T_N columns
                    t_mma = 2.0 * hw.mma_rows * 64 * T_N / hw.peak_flops_per_cycle
                    ec *= t_mma / max(t_mma + hw.convert_exposed_cycles, hw.convert_cycles)
                assert math.isclose(s.ai, ai, rel_tol=1e-12)
                assert math.isclose(s.eff_micro, em, rel_tol=1e-12)
                assert math.isclose(s.eff_core, ec, rel_tol=1e-12)
                perf = model.perf_array(ai, hw.bw_bytes_per_s, ec, hw.peak_flops_per_cycle * hw.clock_hz, hw.n_units)
                assert math.isclose(s.predicted_flops, perf, rel_tol=1e-12)
                c_term = hw.c_buf_bytes * T_MC * T_N
                buf = model.buffer_bytes(T_MA, T_MC, T_K, T_N, hw.a_buf_bytes, hw.b_buf_bytes, 0.0, hw.a_scratch_bytes)
                if 0 < hw.a_unit_cols < T_K:
                    # A is buffered 64 columns deep whatever T_K is: Eq. 1's A terms at that depth, the B term at T_K
                    buf = model.buffer_bytes(T_MA, T_MC, hw.a_unit_cols, T_N, hw.a_buf_bytes, 0.0, 0.0, hw.a_scratch_bytes) + \
                        model.buffer_bytes(T_MA, T_MC, T_K, T_N, 0.0, hw.b_buf_bytes, 0.0, 0.0)
                if hw.acc_capacity_bytes > 0:
                    assert math.isclose(s.buf_bytes_used, buf, rel_tol=1e-12)
                    assert math.isclose(s.acc_bytes_used, c_term, rel_tol=1e-12)
                else:
                    assert math.isclose(s.buf_bytes_used, buf + c_term, rel_tol=1e-12)


def test_select_tiling_orders_and_filters():
    best, scores = atb.atb_select_tiling(8192, 8192, 8192)
    assert atb.atb_tiling_supported(*best)
    assert len(scores) >= 20
    feas = [s for s in scores if s.feasible]
    assert feas and all(a.predicted_flops >= b.predicted_flops for a, b in zip(feas, feas[1:]))
    assert (scores[0].t.T_MA, scores[0].t.T_MC, scores[0].t.T_K, scores[0].t.T_N) == tuple(best)
    for s in scores:                                   # only tilings the kernel accepts are proposed
        assert atb.atb_tiling_supported(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N)
        assert s.predicted_flops <= min(s.mem_bound_flops, s.compute_bound_flops) * (1 + 1e-12)
    # trade-off of Section 5: at fixed (T_MC, T_K, T_N) a larger rho never raises the compute bound,
    # and AI does not depend on T_MA or T_K
    by = {(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N): s for s in scores}
    assert by[(32, 256, 64, 256)].compute_bound_flops < by[(64, 256, 64, 256)].compute_bound_flops \
        < by[(128, 256, 64, 256)].compute_bound_flops
    # slabs of 256 and 128 rows cost the 128-row MMA the same number of switches; the preset's
    # coarse_slab_factor (measured: coarser conversion pipeline) puts the 256-row slab behind, and
    # without it the scores are equal and the smaller buffer goes first
    assert math.isclose(by[(256, 256, 64, 256)].compute_bound_flops,
                        by[(128, 256, 64, 256)].compute_bound_flops * atb.atb_hw_params_b200().coarse_slab_factor, rel_tol=1e-2)
    order = [(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N) for s in scores]
    assert order.index((128, 256, 64, 256)) < order.index((256, 256, 64, 256))
    hw = atb.atb_hw_params_b200()
    hw.coarse_slab_factor = 0.0
    _, flat = atb.atb_select_tiling(8192, 8192, 8192, hw)
    fb = {(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N): s for s in flat}
    assert fb[(128, 256, 64, 256)].predicted_flops == fb[(256, 256, 64, 256)].predicted_flops
    forder = [(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N) for s in flat]
    assert forder.index((128, 256, 64, 256)) < forder.index((256, 256, 64, 256))
    assert by[(32, 256, 64, 256)].ai == by[(256, 256, 64, 256)].ai == by[(32, 256, 128, 256)].ai


def test_select_tiling_small_problem_prefers_more_tiles():
    # 1024 x 1024 has 16 tiles of 256 x 256 on 148 SMs: wave quantisation must show in the score
    best, scores = atb.atb_select_tiling(1024, 1024, 8192)
    big = [s for s in scores if (s.t.T_MC, s.t.T_N) == (256, 256)][0]
    small = [s for s in scores if (s.t.T_MC, s.t.T_N) == (128, 64)][0]
    assert small.compute_bound_flops > big.compute_bound_flops
    assert (best.T_MC, best.T_N) != (256, 256)


def test_b200_refinements_can_be_switched_off():
    """With the refinements at 0 the selection is the paper's Eq. 12 times wave quantisation."""
    hw = atb.atb_hw_params_b200()
    hw.mma_rows = 0; hw.load_latency_cycles = 0.0; hw.pair_efficiency = 0.0; hw.launch_seconds = 0.0
    hw.tile_fixed_cycles = 0.0; hw.drain_cycles_per_column = 0.0; hw.pair_tile_cycles = 0.0; hw.thin_slab_cost = 1.0; hw.coarse_slab_factor = 0.0; hw.deep_kstep_factor = 0.0
    hw.convert_cycles = 0.0; hw.convert_exposed_cycles = 0.0; hw.convert_latency_cycles = 0.0
    _, scores = atb.atb_select_tiling(8192, 8192, 8192, hw)
    for s in scores:
        t = (s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N)
        if (t[1], t[3]) == (256, 512) or t[1:] == (128, 128, 256):
            continue                                   # CTA-pair tilings: scored per CTA with the B tile shared by two
        ref = atb.atb_score_tiling(hw, 8192, t)
        tiles = math.ceil(8192 / t[1]) * math.ceil(8192 / t[3])       # edge tiles compute padding
        useful = 8192 * 8192 / (math.ceil(tiles / 148) * 148 * t[1] * t[3])
        want = min(ref.mem_bound_flops, ref.compute_bound_flops * useful)
        assert math.isclose(s.predicted_flops, want, rel_tol=1e-12), t


def test_select_tiling_errors():
    lib = atb.load_library()
    assert lib.atb_select_tiling(0, 8, 64, None, None, None, None) == 2
    with pytest.raises(atb.AtbError):
        atb.atb_score_tiling(atb.atb_hw_params_b200(), 64, (48, 128, 64, 128))


def test_per_tile_costs():
    """The per-tile terms: every tiling's compute bound grows with K (the fixed cost per output tile
    is spread over more K-steps), the drain term touches only tilings whose accumulator is not
    double-buffered, and the CTA-pair term only CTA-pair tilings."""
    def bounds(K, **kw):
        hw = atb.atb_hw_params_b200()
        for n, v in kw.items():
            setattr(hw, n, v)
        _, scores = atb.atb_select_tiling(8192, 8192, K, hw)
        return {(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N): s.compute_bound_flops for s in scores}
    b1, b4, b16 = bounds(1024), bounds(4096), bounds(16384)
    assert all(b1[t] < b4[t] < b16[t] for t in b1)
    no_drain = bounds(1024, drain_cycles_per_column=0.0)
    for t in b1:
        single = atb.atb_tiling_plan(*t).acc_buffers == 1
        assert (no_drain[t] > b1[t]) == single, t
    no_pair = bounds(1024, pair_tile_cycles=0.0)
    for t in b1:
        assert (no_pair[t] > b1[t]) == ((t[1], t[2], t[3]) == (256, 64, 512)), t
    # shallow K: the CTA-pair tilings (one accumulator of 512 columns to drain per tile) are not chosen
    assert tuple(atb.atb_select_tiling(8192, 8192, 1024)[0])[3] != 512


def test_pair_tilings_are_rated_per_cta_and_chosen_at_deep_k():
    """A CTA of the pair holds half of the 256 x 512 tile: Eq. 1's budgets apply to that half (the whole
    accumulator would not fit one SM's tensor memory).  The pair is measured ahead where K is deep and
    behind where it is shallow (its single accumulator stalls the next tile); there the stacked pair of
    128 x 256 tiles, whose accumulators are double-buffered, is ahead, and the preset follows."""
    best, scores = atb.atb_select_tiling(8192, 8192, 8192, max_scores=256)
    by = {(s.t.T_MA, s.t.T_MC, s.t.T_K, s.t.T_N): s for s in scores}
    pair = by[(128, 256, 64, 512)]
    assert pair.feasible == 1 and pair.acc_bytes_used == 128 * 512 * 4
    assert (best.T_MC, best.T_K, best.T_N) == (256, 64, 512)
    shallow, _ = atb.atb_select_tiling(8192, 8192, 1024)
    assert (shallow.T_MC, shallow.T_K, shallow.T_N) == (128, 128, 256)
    one_row, _ = atb.atb_select_tiling(128, 8192, 8192)          # a single tile row has nothing to share
    assert atb.atb_tiling_plan(*one_row).acc_buffers in (1, 2)

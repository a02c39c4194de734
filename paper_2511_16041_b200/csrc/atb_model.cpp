// Host-side analytical model of Sections 3-5 and the tiling selection built on it.
// Pure host arithmetic in FP64; no CUDA calls.
#include <algorithm>
#include <cmath>
#include <vector>

#include "atb_internal.h"

extern "C" {

void atb_hw_params_b200(atb_hw_params_t* hw) {
    if (!hw) return;
    // Constants fitted to measured throughput of atb_gemm on B200: every supported tiling on 15
    // shapes (cubes, shallow and deep K, FFN-like and odd sizes) and 6 tilings on 125 shapes.  The
    // fit maximises what the selection is for - the measured rate of the tiling it picks against the
    // best measured one (paper_2511_16041_b200/calibrate.py repeats the fit on the GPU at hand and
    // prints that figure).  They are a fit, not the paper's model: the terms beyond Eq. 1, 2, 12-15 are
    // named in atb_hw_params_t and each can be switched off.
    // One unit = one SM.  Dense BF16 tcgen05 peak: 8192 FLOP per cycle per SM; the clock is the one
    // a tensor-bound kernel settles at under the 1 kW power cap (1.65 PFLOP/s over 148 SMs).
    hw->peak_flops_per_cycle = 8192.0;
    hw->clock_hz = 1.361e9;
    hw->n_units = 148;
    // Eq. 2 / Eq. 12 with the physical byte costs of the operands (BFP16 A 9/8 B, BF16 B and C 2 B): AI is
    // FLOP per byte of tile traffic, which on B200 flows L2 -> SM (ncu: 163.8 FLOP/B at 256 x 256, the
    // formula's value).  The bandwidth is the L2 -> SM feed rate of 148 SMs; it is FITTED (no direct
    // measurement; the kernels have been seen to draw 9.2 TB/s without being bound by it).
    hw->bw_bytes_per_s = 14.0e12;
    hw->a_bytes = 1.125; hw->b_bytes = 2.0; hw->c_bytes = 2.0;
    // Eq. 1, A and B terms, against shared memory: raw BFP16 slabs double-buffered at 9/8 B, two
    // dequantised BF16 copies per slab row (the "converted copy" of Table 2), B double-buffered.
    // The C term is budgeted against TMEM (128 lanes x 512 columns x 4 B) instead.
    hw->a_buf_bytes = 1.125; hw->b_buf_bytes = 2.0; hw->c_buf_bytes = 4.0;
    hw->a_scratch_bytes = 2.0 * 2.0;
    hw->buf_capacity_bytes = 227.0 * 1024.0;
    hw->acc_capacity_bytes = 128.0 * 512.0 * 4.0;
    hw->share_rows = 1; hw->share_cols = 1;
    // Eq. 13: one UMMA covers K = 16 -> eta = 1/16 instructions per unit of T_K, II = 1.
    hw->eta = 1.0 / 16.0; hw->eps_cycles = 0.05; hw->ii = 1.0;
    hw->delta_cycles = 20.0;                  // per-slab hand-over (barrier round trip, commit) left once the conversion has its own term
    hw->mma_rows = 128;
    hw->load_latency_cycles = 1200.0;
    hw->pair_efficiency = 1.0;
    hw->launch_seconds = 1.0e-5;
    hw->tile_fixed_cycles = 1000.0;
    hw->drain_cycles_per_column = 2.0;
    hw->pair_tile_cycles = 4000.0;
    hw->thin_slab_cost = 0.3;                 // measured: a bundled slab costs about 0.3 of a switch (rho = 4 reaches 0.97, rho = 8 0.87 of rho = 2)
    hw->coarse_slab_factor = 0.92;            // 256-row slabs: measured 0.87-0.92 of 128-row slabs
    hw->deep_kstep_factor = 0.0;              // retired: T_K = 128 runs level with T_K = 64 where the rings are as deep
    // The conversion of A, on the compute side.  Measured against the same pipeline without it the
    // conversion costs 8 % at T_N = 256 and 3.5 % on the CTA pair (a unit feeds 512 columns there): about
    // 45 cycles per unit that the UMMAs do not hide; at T_N <= 128 the 16 dequantiser warps bind at
    // about 400 cycles per unit.  A converted-operand ring of n units hides a conversion latency of about
    // 700 cycles only if n * t_mma covers it (two groups instead of four measured -15...-20 %).
    hw->convert_cycles = 400.0;
    hw->convert_exposed_cycles = 45.0;
    hw->convert_latency_cycles = 700.0;
    hw->a_unit_cols = 64;                     // raw slabs of T_MA x 64 and converted groups of 128 x 64 for every T_K
}

void atb_hw_params_xdna2(atb_hw_params_t* hw, int precision_config) {
    if (!hw) return;
    hw->peak_flops_per_cycle = 1024.0;        // 512 MAC per cycle per core (Section 2.4)
    hw->clock_hz = 1.8e9;
    hw->n_units = 32;
    hw->bw_bytes_per_s = 65e9;                // Section 5
    hw->buf_capacity_bytes = 63.0 * 1024.0;   // Eq. 3
    hw->acc_capacity_bytes = 0.0;             // C lives in the same L1
    hw->share_rows = 4; hw->share_cols = 8;   // Eq. 2
    hw->eta = 1.0 / 8.0; hw->eps_cycles = 20.0; hw->ii = 1.0;
    hw->delta_cycles = 50.0;                  // Section 5
    hw->a_scratch_bytes = 0.0;
    hw->mma_rows = 0; hw->load_latency_cycles = 0.0; hw->pair_efficiency = 0.0; hw->launch_seconds = 0.0;
    hw->tile_fixed_cycles = 0.0; hw->drain_cycles_per_column = 0.0; hw->pair_tile_cycles = 0.0;
    hw->thin_slab_cost = 1.0; hw->coarse_slab_factor = 0.0; hw->deep_kstep_factor = 0.0;
    hw->convert_cycles = 0.0; hw->convert_exposed_cycles = 0.0; hw->convert_latency_cycles = 0.0;
    hw->a_unit_cols = 0;
    switch (precision_config) {
        case 1:   // A, C in BF16, B in BFP16 (text: 1.25 B in AI; 9/8 B reproduces the buffer column)
            hw->a_bytes = 2.0; hw->b_bytes = 1.25; hw->c_bytes = 2.0;
            hw->a_buf_bytes = 2.0; hw->b_buf_bytes = 1.125; hw->c_buf_bytes = 2.0;
            hw->a_scratch_bytes = 1.125;      // one BFP16-converted copy of the A slab
            break;
        case 3:   // all BFP16, BF16 accumulation
            hw->a_bytes = hw->b_bytes = hw->c_bytes = 1.25;
            hw->a_buf_bytes = hw->b_buf_bytes = 1.125; hw->c_buf_bytes = 2.125;
            break;
        default:  // 2: all BFP16
            hw->a_bytes = hw->b_bytes = hw->c_bytes = 1.25;
            hw->a_buf_bytes = hw->b_buf_bytes = hw->c_buf_bytes = 1.125;
            break;
    }
}

atb_status_t atb_score_tiling(const atb_hw_params_t* hw, int64_t K, atb_tiling_t t, atb_tiling_score_t* out) {
    atb::clear_error();
    if (!hw || !out) return atb::fail(ATB_ERR_NULL_POINTER, "hw and out must be non-NULL");
    if (t.T_MA <= 0 || t.T_MC <= 0 || t.T_K <= 0 || t.T_N <= 0 || t.T_MC % t.T_MA != 0 || K <= 0)
        return atb::fail(ATB_ERR_BAD_TILING, "need positive sizes and T_MC a multiple of T_MA");
    const double rho = static_cast<double>(t.T_MC) / t.T_MA;
    const double TMC = t.T_MC, TK = t.T_K, TN = t.T_N, TMA = t.T_MA;
    out->t = t;
    // Eq. 1 (left-hand side), with the optional converted-copy term.
    const double TKA = (hw->a_unit_cols > 0 && hw->a_unit_cols < t.T_K) ? hw->a_unit_cols : TK;   // depth of an A buffer
    const double ab = (2.0 * hw->a_buf_bytes / rho) * TMC * TKA + 2.0 * hw->b_buf_bytes * TK * TN +
                      hw->a_scratch_bytes * TMA * TKA;
    const double cb = hw->c_buf_bytes * TMC * TN;
    if (hw->acc_capacity_bytes > 0.0) {
        out->buf_bytes_used = ab;
        out->acc_bytes_used = cb;
        out->feasible = (ab <= hw->buf_capacity_bytes && cb <= hw->acc_capacity_bytes) ? 1 : 0;
    } else {
        out->buf_bytes_used = ab + cb;
        out->acc_bytes_used = cb;
        out->feasible = (ab + cb <= hw->buf_capacity_bytes) ? 1 : 0;
    }
    // Eq. 2
    out->ai = 2.0 / (hw->a_bytes / (hw->share_cols * TN) + hw->b_bytes / (hw->share_rows * TMC) +
                     hw->c_bytes / static_cast<double>(K));
    // Eq. 13, Eq. 15
    out->eff_micro = hw->eta * TK / (hw->eps_cycles + hw->eta * hw->ii * TK);
    double rho_eff = rho;
    if (hw->mma_rows > 0) {
        const double per_mma = TMC / hw->mma_rows;      // switches if every slab were one MMA operand
        if (t.T_MA > hw->mma_rows) rho_eff = per_mma;
        else if (t.T_MA < hw->mma_rows && per_mma >= 1.0) rho_eff = per_mma + (rho - per_mma) * hw->thin_slab_cost;
    }
    out->eff_core = 1.0 / (1.0 / out->eff_micro +
                           hw->delta_cycles * rho_eff * hw->peak_flops_per_cycle / (2.0 * TMC * TN * TK));
    if (hw->mma_rows > 0 && t.T_MA > hw->mma_rows && hw->coarse_slab_factor > 0.0) out->eff_core *= hw->coarse_slab_factor;
    if (hw->mma_rows > 0 && t.T_K > 64 && hw->deep_kstep_factor > 0.0) out->eff_core *= hw->deep_kstep_factor;
    if (hw->mma_rows > 0 && (hw->convert_cycles > 0.0 || hw->convert_exposed_cycles > 0.0)) {
        const double t_mma = 2.0 * hw->mma_rows * 64.0 * TN / hw->peak_flops_per_cycle;
        out->eff_core *= t_mma / std::max(t_mma + hw->convert_exposed_cycles, hw->convert_cycles);
    }
    // Eq. 12
    out->mem_bound_flops = out->ai * hw->bw_bytes_per_s;
    out->compute_bound_flops = out->eff_core * hw->peak_flops_per_cycle * hw->clock_hz * hw->n_units;
    out->predicted_flops = std::min(out->mem_bound_flops, out->compute_bound_flops);
    return ATB_OK;
}

atb_status_t atb_select_tiling(int64_t M, int64_t N, int64_t K, const atb_hw_params_t* hw_in,
                               atb_tiling_t* best, atb_tiling_score_t* scores, int* n_scores) {
    atb::clear_error();
    if (M < 1 || N < 1 || K < 1) return atb::fail(ATB_ERR_BAD_SHAPE, "M, N, K must be positive");
    if ((scores == nullptr) != (n_scores == nullptr))
        return atb::fail(ATB_ERR_NULL_POINTER, "scores and n_scores go together");
    atb_hw_params_t hw;
    if (hw_in) hw = *hw_in; else atb_hw_params_b200(&hw);

    static const int kMC[] = {128, 256, 384}, kN[] = {64, 128, 256, 512}, kK[] = {64, 128}, kMA[] = {32, 64, 128, 256};
    std::vector<atb_tiling_score_t> all;
    for (int mc : kMC) for (int n : kN) for (int k : kK) for (int ma : kMA) {
        atb::GemmPlan plan;
        // two stacked 128 x 256 tiles on a CTA pair (where M has more than one tile row), else single CTAs
        const bool stacked = atb::is_stacked_pair_tiling(mc, k, n) && M > 128;
        if (ma > mc || !atb::plan_gemm(ma, mc, k, n, &plan, !stacked)) continue;
        const bool pair = atb::is_pair_tiling(mc, k, n);
        atb_hw_params_t h = hw;
        if (pair || stacked) h.share_rows = hw.share_rows * 2;      // the B tile is shared by the two CTAs (Eq. 2)
        // thin slabs get the bundle discount only as far as this tiling's raw ring lets them be bundled
        const int slab = ma;
        if (hw.mma_rows > 0 && slab < hw.mma_rows) {
            const int spg = hw.mma_rows / slab, b = atb::slab_bundle(spg, plan.n_raw_stages, plan.dq_groups);
            const double full = static_cast<double>(spg) / b;              // full switches per operand group
            h.thin_slab_cost = ((full - 1.0) + (spg - full) * hw.thin_slab_cost) / (spg - 1.0);
        }
        atb_tiling_score_t s;
        if (atb_score_tiling(&h, K, atb_tiling_t{ma, mc, k, n}, &s) != ATB_OK) continue;
        if (pair) {
            // each CTA of the pair runs Eq. 13-15 on its own 128 rows
            atb_tiling_score_t half;
            atb_score_tiling(&h, K, atb_tiling_t{ma, 128, k, n}, &half);
            s.eff_core = half.eff_core;
            s.compute_bound_flops = half.compute_bound_flops;
            // ... and holds its own half of the tile: Eq. 1's budgets are per CTA
            s.feasible = half.feasible;
            s.buf_bytes_used = half.buf_bytes_used;
            s.acc_bytes_used = half.acc_bytes_used;
            if (hw.pair_efficiency > 0.0) s.compute_bound_flops *= hw.pair_efficiency;
        }
        if (stacked && hw.pair_efficiency > 0.0) s.compute_bound_flops *= hw.pair_efficiency;
        // Look-ahead of the B ring (Little's law on the buffer of Eq. 1): a stage is busy from the
        // moment its load is issued until its UMMAs have run, so n stages sustain at most
        // n * t_stage / (latency + t_stage) of the UMMA rate.
        if (hw.load_latency_cycles > 0.0) {
            const double rows_per_unit = pair ? 128.0 : mc;
            const double kstep_cycles = 2.0 * rows_per_unit * n * k / hw.peak_flops_per_cycle;
            const double sustain = plan.n_b_stages * kstep_cycles / (hw.load_latency_cycles + kstep_cycles);
            if (sustain < 1.0) s.compute_bound_flops *= sustain;
        }
        // Look-ahead of the converted-operand ring, the same law: n units of t_mma cycles each hide the
        // conversion latency only if n * t covers it.
        if (hw.convert_latency_cycles > 0.0 && hw.mma_rows > 0) {
            const double t_mma = 2.0 * hw.mma_rows * 64.0 * n / hw.peak_flops_per_cycle;
            const double t_unit = std::max(t_mma + hw.convert_exposed_cycles, hw.convert_cycles);
            const double sustain = plan.n_groups * t_unit / (hw.convert_latency_cycles + t_unit);
            if (sustain < 1.0) s.compute_bound_flops *= sustain;
        }
        // Per-tile costs that the K loop does not hide: filling the rings, and - with a single
        // accumulator in TMEM - the UMMAs idling while the epilogue drains it.
        {
            const double rows_per_unit = pair ? 128.0 : mc;
            const double kstep_cycles = 2.0 * rows_per_unit * n * k / (hw.peak_flops_per_cycle * s.eff_core);
            const double k_steps = std::ceil(static_cast<double>(K) / k);
            const double acc_cols = rows_per_unit / 128.0 * n;                  // FP32 columns per unit
            double tile_cycles = hw.tile_fixed_cycles + (pair ? hw.pair_tile_cycles : 0.0);
            if (plan.acc_bufs < 2) tile_cycles += hw.drain_cycles_per_column * acc_cols;
            s.compute_bound_flops *= k_steps * kstep_cycles / (k_steps * kstep_cycles + tile_cycles);
        }
        // Wave quantisation: tiles are spread over the units (pairs of units for pair tilings); the
        // last wave may be partly empty and edge tiles compute padding.
        const double units = (pair || stacked) ? hw.n_units / 2 : hw.n_units;
        const double tile_rows = stacked ? 2.0 * mc : mc;                  // rows a unit (CTA or pair) covers at a time
        const double tiles = std::ceil(static_cast<double>(M) / tile_rows) * static_cast<double>(atb::ceil_div(N, n));
        const double waves = std::ceil(tiles / units);
        const double useful = (static_cast<double>(M) * N) / (waves * units * tile_rows * n);
        s.compute_bound_flops *= useful;
        s.predicted_flops = std::min(s.mem_bound_flops, s.compute_bound_flops);
        if (hw.launch_seconds > 0.0) {
            const double flop = 2.0 * M * N * K;
            s.predicted_flops = flop / (flop / s.predicted_flops + hw.launch_seconds);
        }
        all.push_back(s);
    }
    std::stable_sort(all.begin(), all.end(), [](const atb_tiling_score_t& x, const atb_tiling_score_t& y) {
        if (x.feasible != y.feasible) return x.feasible > y.feasible;
        // equal predictions: the smaller A buffer first - asymmetric buffering costs nothing there
        if (x.predicted_flops != y.predicted_flops) return x.predicted_flops > y.predicted_flops;
        return x.t.T_MA < y.t.T_MA;
    });
    if (all.empty() || !all.front().feasible) return atb::fail(ATB_ERR_BAD_SHAPE, "no supported tiling is feasible");
    if (best) *best = all.front().t;
    if (scores) {
        const int cap = *n_scores;
        if (cap < 0) return atb::fail(ATB_ERR_BUFFER_TOO_SMALL, "negative capacity");
        const int n = std::min<int>(cap, static_cast<int>(all.size()));
        for (int i = 0; i < n; ++i) scores[i] = all[i];
        *n_scores = n;
    }
    return ATB_OK;
}

}  // extern "C"

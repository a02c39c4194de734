"""The paper's analytical model, written out formula by formula.  TEST INFRASTRUCTURE ONLY.

Plain Python floats (FP64), one function per displayed formula, in the paper's
notation.  The product's host-side planner (``atb_select_tiling``) is a separate
C++ implementation; the tests compare the two.  Pins: the arithmetic columns of
Table 2 and the worked T_load example of Section 4.1 (``tests/golden``); closed
forms and monotonic trends of Sections 3 and 5.  Numerical agreement of
Eff_core with Table 1 is unpinned (the paper claims trends only).
"""
from __future__ import annotations

import math


def ai_rho(T_MC, T_N, K, a, b, c):
    """Arithmetic intensity of one output tile, unnumbered display of Section 3.1:
    AI_rho = 2 / (a/T_N + b/T_MC + c/K); independent of T_K and rho."""
    return 2.0 / (a / T_N + b / T_MC + c / K)


def buffer_bytes(T_MA, T_MC, T_K, T_N, a, b, c, a_scratch=0.0):
    """Left-hand side of Eq. 1: A and B double-buffered, C single-buffered,
    (2a/rho) T_MC T_K + 2b T_K T_N + c T_MC T_N.

    ``a_scratch`` adds one single-buffered converted copy of the A slab,
    a_scratch * T_MA * T_K bytes; Table 2's Config-1 buffer column is only
    reproduced with it (the converted copy is implied by Section 4.3's remark
    that BFP16<->BF16 conversions take place inside the kernel)."""
    rho = T_MC / T_MA
    return (2.0 * a / rho) * T_MC * T_K + 2.0 * b * T_K * T_N + c * T_MC * T_N \
        + a_scratch * T_MA * T_K


def ai_array(T_MC, T_N, K, a, b, c, n_row=4, n_col=8):
    """Eq. 2: the array-level tile is n_row*T_MC by n_col*T_N (A broadcast across
    columns, B across rows)."""
    return 2.0 / (a / (n_col * T_N) + b / (n_row * T_MC) + c / K)


def t_load(latencies, counts, U_LD):
    """Eq. 5: lower bound of the prolog.  Instruction types sorted by descending
    latency; S_(i) = cumulative load count; max_i (l_(i) + ceil(S_(i)/U_LD) - 1)."""
    order = sorted(range(len(latencies)), key=lambda i: -latencies[i])
    best, cum = 0, 0
    for i in order:
        cum += counts[i]
        best = max(best, latencies[i] + math.ceil(cum / U_LD) - 1)
    return best


def eff_micro(T_K, eta, eps, II):
    """Eq. 13: eta T_K / (eps + eta II T_K); saturates at 1/II."""
    return eta * T_K / (eps + eta * II * T_K)


def t_asym(T_MA, T_MC, T_K, T_N, K, peak, effm, delta):
    """Eq. 14 (peak in FLOP per cycle, delta in cycles): compute time of one
    output tile plus rho*K/T_K slab switches of delta cycles each."""
    rho = T_MC / T_MA
    return 2.0 * T_MC * K * T_N / (peak * effm) + delta * rho * K / T_K


def eff_core(T_MA, T_MC, T_K, T_N, peak, effm, delta):
    """Eq. 15: 1 / (1/Eff_micro + delta rho peak / (2 T_MC T_N T_K))."""
    rho = T_MC / T_MA
    return 1.0 / (1.0 / effm + delta * rho * peak / (2.0 * T_MC * T_N * T_K))


def perf_array(ai, bw, effc, peak_core_flops, n_core):
    """Eq. 12: min(AI * BW_offchip, Eff_core * Perf_core_peak * N_core), FLOP/s."""
    return min(ai * bw, effc * peak_core_flops * n_core)

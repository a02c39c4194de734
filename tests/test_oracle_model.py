"""Pins for the oracle's restatement of the analytical model (Sections 3-5)."""
import math
import os

import pytest

from oracle import model

HERE = os.path.dirname(os.path.abspath(__file__))

# Per-element byte costs (A, B, C).  The AI column of Table 2 uses the text's 1.25 B per
# BFP16 element (Section 3.1); the buffer column is only reproduced with the format's true
# 9/8 B (Section 2.4).  Config 1: A, C in BF16, B in BFP16, plus a single converted copy of
# the A slab; Config 2: all BFP16; Config 3: all BFP16 with a 2.125 B accumulator/output tile.
AI_BYTES = {"C1": (2.0, 1.25, 2.0), "C2": (1.25, 1.25, 1.25), "C3": (1.25, 1.25, 1.25)}
BUF_BYTES = {"C1": (2.0, 1.125, 2.0, 1.125), "C2": (1.125, 1.125, 1.125, 0.0),
             "C3": (1.125, 1.125, 2.125, 0.0)}


def rows():
    out = []
    with open(os.path.join(HERE, "golden", "table2_model_columns.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            t = line.split()
            out.append(dict(cfg=t[0], K=int(t[1]), T_MC=int(t[2]), T_K=int(t[3]), T_N=int(t[4]),
                            rho=int(t[5]), buf=t[6], buf1=t[7], perf_core=float(t[8]),
                            compute=float(t[9]), ai=float(t[10]), mem=float(t[11]),
                            measured=float(t[12])))
    return out


def _printed(value, printed_text):
    """value agrees with a printed figure to the digits printed (half a unit of the last place)."""
    digits = len(printed_text.split(".")[1]) if "." in printed_text else 0
    return abs(value - float(printed_text)) <= 0.5 * 10 ** -digits + 1e-9


@pytest.mark.parametrize("r", rows(), ids=lambda r: f"{r['cfg']}-{r['T_MC']}x{r['T_K']}x{r['T_N']}-rho{r['rho']}")
def test_table2_row(r):
    a, b, c = AI_BYTES[r["cfg"]]
    ai = model.ai_array(r["T_MC"], r["T_N"], r["K"], a, b, c, n_row=4, n_col=8)
    assert abs(ai - r["ai"]) <= 0.5
    mem = ai * 65e9 / 1e12
    assert abs(mem - r["mem"]) <= 0.075           # one printed decimal; 14.04 is printed as 14.1
    assert abs(r["perf_core"] * 32 - r["compute"]) <= 0.17      # Perf_core is printed to 2 digits
    bound = model.perf_array(ai, 65e9, r["perf_core"] / 1.84, 1.84e12, 32) / 1e12
    assert r["measured"] <= bound * 1.001         # Eq. 12 bounds what was measured
    if r["buf"] != "-":
        ba, bb, bc, bs = BUF_BYTES[r["cfg"]]
        T_MA = r["T_MC"] // r["rho"]
        used = model.buffer_bytes(T_MA, r["T_MC"], r["T_K"], r["T_N"], ba, bb, bc, bs) / 1024
        sym = model.buffer_bytes(r["T_MC"], r["T_MC"], r["T_K"], r["T_N"], ba, bb, bc, bs) / 1024
        assert _printed(used, r["buf"]), used
        assert _printed(sym, r["buf1"]) or abs(sym - float(r["buf1"])) <= 0.5, sym
        assert used <= 63.0                        # Eq. 3: fits the 63 KB of usable L1
        if r["rho"] > 1:
            assert sym > 63.0                      # ... and would not fit without ATB


def test_t_load_worked_example():
    # Section 4.1: three instruction types of latency 3, counts n_C=2, n_A=n_B=1, two load slots
    assert model.t_load([3, 3, 3], [2, 1, 1], 2) == 4
    assert model.t_load([3], [1], 2) == 3
    assert model.t_load([8, 3], [2, 4], 2) == 8       # long loads first, short ones hide behind them
    assert model.t_load([8, 3], [2, 14], 2) == 3 + 8 - 1


def test_ai_closed_forms():
    # K -> infinity: 2/(a/T_N + b/T_MC); independent of T_K and rho by construction
    assert math.isclose(model.ai_rho(256, 256, 1e18, 1.125, 2, 2), 2 / (1.125 / 256 + 2 / 256))
    # symmetric square tile with equal byte costs: AI = 2 / (2a/T + a/K)
    assert math.isclose(model.ai_rho(64, 64, 64, 2, 2, 2), 2 / (3 * 2 / 64))
    # monotone in T_MC and T_N
    assert model.ai_rho(256, 128, 4096, 1, 2, 2) > model.ai_rho(128, 128, 4096, 1, 2, 2)
    assert model.ai_rho(128, 256, 4096, 1, 2, 2) > model.ai_rho(128, 128, 4096, 1, 2, 2)
    # n_row = n_col = 1 reduces the array form to the single-core form
    assert model.ai_array(128, 64, 512, 1, 2, 3, 1, 1) == model.ai_rho(128, 64, 512, 1, 2, 3)


def test_buffer_closed_forms():
    # rho = 1 is the symmetric cost 2a T_M T_K + 2b T_K T_N + c T_M T_N
    assert model.buffer_bytes(64, 64, 32, 16, 1, 2, 4) == 2 * 64 * 32 + 2 * 2 * 32 * 16 + 4 * 64 * 16
    # the A term shrinks by rho, the others do not
    full = model.buffer_bytes(128, 128, 64, 128, 2, 1, 2)
    quarter = model.buffer_bytes(32, 128, 64, 128, 2, 1, 2)
    assert full - quarter == 2 * 2 * (128 - 32) * 64


def test_efficiency_forms_and_trends():
    eta, eps, II, peak, delta = 1 / 8, 20.0, 1.0, 1024.0, 50.0
    # saturation of Eq. 13 at 1/II, linear growth for small T_K
    assert math.isclose(model.eff_micro(1e12, eta, eps, II), 1 / II, rel_tol=1e-9)
    assert math.isclose(model.eff_micro(1e-6, eta, eps, II), eta * 1e-6 / eps, rel_tol=1e-6)
    for T_K in (8, 16, 32, 64):
        em = model.eff_micro(T_K, eta, eps, II)
        prev = None
        for rho in (1, 2, 4, 8):
            ec = model.eff_core(128 // rho, 128, T_K, 128, peak, em, delta)
            # Eq. 15 is Eq. 14 re-arranged
            ta = model.t_asym(128 // rho, 128, T_K, 128, 4096, peak, em, delta)
            assert math.isclose(ec, 2 * 128 * 4096 * 128 / ta / peak, rel_tol=1e-12)
            assert ec < em                         # switching only costs
            if prev is not None:
                assert ec < prev                   # Table 1: falls with rho at fixed T_K
            prev = ec
        assert math.isclose(model.eff_core(128, 128, T_K, 128, peak, em, 0.0), em)   # delta -> 0
    # rises with T_K at fixed rho, and the relative loss rho=1 -> 8 shrinks with T_K (Table 1)
    loss = []
    for T_K in (8, 16, 32, 64):
        em = model.eff_micro(T_K, eta, eps, II)
        e1 = model.eff_core(128, 128, T_K, 128, peak, em, delta)
        e8 = model.eff_core(16, 128, T_K, 128, peak, em, delta)
        loss.append(1 - e8 / e1)
    assert loss == sorted(loss, reverse=True)
    effs = [model.eff_core(32, 128, T_K, 128, peak, model.eff_micro(T_K, eta, eps, II), delta)
            for T_K in (8, 16, 32, 64)]
    assert effs == sorted(effs)


def test_perf_array_is_min_of_bounds():
    assert model.perf_array(100.0, 65e9, 0.5, 1.84e12, 32) == 100.0 * 65e9
    assert model.perf_array(1000.0, 65e9, 0.5, 1.84e12, 32) == 0.5 * 1.84e12 * 32

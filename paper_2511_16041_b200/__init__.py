"""Python binding of ``libatb.so`` - the asymmetric-tile-buffered BFP16 x BF16 GEMM for B200.

Argument marshalling only: every step of the hot path (quantisation, dequantisation, the
GEMM, the epilogue) runs in the CUDA kernels behind the C ABI declared in ``include/atb.h``.
The functions carry the C names.  PyTorch is used for device memory and streams.

There is no CPU path: importing works anywhere (the input generators in
``paper_2511_16041_b200.inputs`` need only numpy), but the first call of a device function
raises if the library cannot be loaded.
"""
from __future__ import annotations

import ctypes
import os
from typing import NamedTuple

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("ATB_LIBRARY_PATH") or os.path.join(_HERE, "libatb.so")
_lib = None

ATB_OK = 0
STATUS_NAMES = {
    0: "ATB_OK", 1: "ATB_ERR_NULL_POINTER", 2: "ATB_ERR_BAD_SHAPE", 3: "ATB_ERR_BAD_TILING",
    4: "ATB_ERR_MISALIGNED", 5: "ATB_ERR_UNSUPPORTED_DEVICE", 6: "ATB_ERR_CUDA",
    7: "ATB_ERR_BUFFER_TOO_SMALL", 8: "ATB_ERR_DEVICE_TIMEOUT",
}


class AtbError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"{STATUS_NAMES.get(status, status)}: {message}")
        self.status = status


class atb_tiling_t(ctypes.Structure):
    _fields_ = [("T_MA", ctypes.c_int), ("T_MC", ctypes.c_int), ("T_K", ctypes.c_int), ("T_N", ctypes.c_int)]


class atb_hw_params_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_double) for n in ("peak_flops_per_cycle", "clock_hz")] + [("n_units", ctypes.c_int)] + \
               [(n, ctypes.c_double) for n in ("bw_bytes_per_s", "a_bytes", "b_bytes", "c_bytes", "a_buf_bytes",
                                               "b_buf_bytes", "c_buf_bytes", "a_scratch_bytes",
                                               "buf_capacity_bytes", "acc_capacity_bytes")] + \
               [("share_rows", ctypes.c_int), ("share_cols", ctypes.c_int)] + \
               [(n, ctypes.c_double) for n in ("eta", "eps_cycles", "ii", "delta_cycles")] + \
               [("mma_rows", ctypes.c_int)] + \
               [(n, ctypes.c_double) for n in ("load_latency_cycles", "pair_efficiency", "launch_seconds", "tile_fixed_cycles",
                                               "drain_cycles_per_column", "pair_tile_cycles", "thin_slab_cost",
                                               "coarse_slab_factor", "deep_kstep_factor", "convert_cycles",
                                               "convert_exposed_cycles", "convert_latency_cycles")] + \
               [("a_unit_cols", ctypes.c_int)]


class atb_tiling_score_t(ctypes.Structure):
    _fields_ = [("t", atb_tiling_t), ("feasible", ctypes.c_int)] + \
               [(n, ctypes.c_double) for n in ("buf_bytes_used", "acc_bytes_used", "ai", "eff_micro", "eff_core",
                                               "mem_bound_flops", "compute_bound_flops", "predicted_flops")]


class atb_plan_t(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int) for n in ("n_b_stages", "n_raw_stages", "n_a_groups", "dequant_groups",
                                            "acc_buffers", "tmem_columns", "smem_bytes")]


class Tiling(NamedTuple):
    T_MA: int
    T_MC: int
    T_K: int
    T_N: int


EXPORTED_SYMBOLS = [
    "atb_status_string", "atb_last_error_message", "atb_bfp16_mant_bytes", "atb_bfp16_exp_bytes",
    "atb_quantize_bfp16", "atb_gemm", "atb_gemm_bfp16_out", "atb_gemm_config", "atb_gemm_config_tiled", "atb_gemm_splitk", "atb_gemm_splitk_workspace_bytes", "atb_select_splits",
    "atb_gemm_splitk_noalloc",
    "atb_tiling_supported", "atb_tiling_plan", "atb_device_status",
    "atb_hw_params_b200", "atb_hw_params_xdna2", "atb_score_tiling", "atb_select_tiling",
]


def load_library():
    """Loads ``libatb.so`` (built in-tree by ``_build.build_library``).  Raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -m paper_2511_16041_b200._build` (there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    i64, vp, ci = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int
    lib.atb_status_string.restype = ctypes.c_char_p
    lib.atb_status_string.argtypes = [ci]
    lib.atb_last_error_message.restype = ctypes.c_char_p
    lib.atb_bfp16_mant_bytes.restype = ctypes.c_size_t
    lib.atb_bfp16_mant_bytes.argtypes = [i64, i64]
    lib.atb_bfp16_exp_bytes.restype = ctypes.c_size_t
    lib.atb_bfp16_exp_bytes.argtypes = [i64, i64]
    lib.atb_quantize_bfp16.restype = ci
    lib.atb_quantize_bfp16.argtypes = [vp, i64, i64, i64, vp, vp, vp]
    lib.atb_gemm.restype = ci
    lib.atb_gemm.argtypes = [i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, i64, vp, i64, vp]
    lib.atb_gemm_bfp16_out.restype = ci
    lib.atb_gemm_bfp16_out.argtypes = [i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, i64, vp, vp, vp]
    lib.atb_gemm_config.restype = ci
    lib.atb_gemm_config.argtypes = [ci, i64, i64, i64, vp, vp, i64, vp, vp, vp, vp, i64, vp]
    lib.atb_gemm_config_tiled.restype = ci
    lib.atb_gemm_config_tiled.argtypes = [ci, i64, i64, i64, ci, ci, ci, ci, vp, vp, i64, vp, vp, vp, vp, i64, vp]
    lib.atb_gemm_splitk.restype = ci
    lib.atb_gemm_splitk.argtypes = [i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, i64, vp, i64, ci, vp, ctypes.c_size_t, vp]
    lib.atb_gemm_splitk_noalloc.restype = ci
    lib.atb_gemm_splitk_noalloc.argtypes = [i64, i64, i64, ci, ci, ci, ci, vp, vp, vp, i64, vp, i64, ci, vp]
    lib.atb_gemm_splitk_workspace_bytes.restype = ctypes.c_size_t
    lib.atb_gemm_splitk_workspace_bytes.argtypes = [i64, i64, ci, ci]
    lib.atb_select_splits.restype = ci
    lib.atb_select_splits.argtypes = [i64, i64, i64, ci, ci, ci]
    lib.atb_tiling_supported.restype = ci
    lib.atb_tiling_supported.argtypes = [ci, ci, ci, ci]
    lib.atb_tiling_plan.restype = ci
    lib.atb_tiling_plan.argtypes = [ci, ci, ci, ci, ctypes.POINTER(atb_plan_t)]
    lib.atb_device_status.restype = ci
    lib.atb_device_status.argtypes = [vp]
    lib.atb_hw_params_b200.restype = None
    lib.atb_hw_params_b200.argtypes = [ctypes.POINTER(atb_hw_params_t)]
    lib.atb_hw_params_xdna2.restype = None
    lib.atb_hw_params_xdna2.argtypes = [ctypes.POINTER(atb_hw_params_t), ci]
    lib.atb_score_tiling.restype = ci
    lib.atb_score_tiling.argtypes = [ctypes.POINTER(atb_hw_params_t), i64, atb_tiling_t,
                                     ctypes.POINTER(atb_tiling_score_t)]
    lib.atb_select_tiling.restype = ci
    lib.atb_select_tiling.argtypes = [i64, i64, i64, ctypes.POINTER(atb_hw_params_t),
                                      ctypes.POINTER(atb_tiling_t), ctypes.POINTER(atb_tiling_score_t),
                                      ctypes.POINTER(ci)]
    _lib = lib
    return lib


def _check(status: int):
    if status != ATB_OK:
        raise AtbError(status, load_library().atb_last_error_message().decode())


def _stream_ptr(stream):
    if stream is None:
        import torch
        return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    if isinstance(stream, int):
        return ctypes.c_void_p(stream)
    return ctypes.c_void_p(stream.cuda_stream)


def _dev_ptr(t):
    return ctypes.c_void_p(t if isinstance(t, int) else t.data_ptr())


# ------------------------------------------------------------------ plain helpers
def atb_status_string(status: int) -> str:
    return load_library().atb_status_string(status).decode()


def atb_last_error_message() -> str:
    return load_library().atb_last_error_message().decode()


def atb_bfp16_mant_bytes(M: int, K: int) -> int:
    return int(load_library().atb_bfp16_mant_bytes(M, K))


def atb_bfp16_exp_bytes(M: int, K: int) -> int:
    return int(load_library().atb_bfp16_exp_bytes(M, K))


def atb_tiling_supported(T_MA: int, T_MC: int, T_K: int, T_N: int) -> bool:
    return bool(load_library().atb_tiling_supported(T_MA, T_MC, T_K, T_N))


def atb_tiling_plan(T_MA: int, T_MC: int, T_K: int, T_N: int) -> atb_plan_t:
    plan = atb_plan_t()
    _check(load_library().atb_tiling_plan(T_MA, T_MC, T_K, T_N, ctypes.byref(plan)))
    return plan


# ------------------------------------------------------------------ device calls
def atb_quantize_bfp16(A, mant=None, exp=None, stream=None):
    """fp32 CUDA tensor ``A[M][K]`` (row stride = lda) -> (mant int8 [M][K], exponent plane uint8).

    The exponent plane is the flat device layout ``[ceil(K/64)][roundup(M,32)][8]``."""
    import torch
    assert A.is_cuda and A.dtype == torch.float32 and A.dim() == 2 and A.stride(1) == 1
    M, K = A.shape
    if mant is None:
        mant = torch.empty((M, K), dtype=torch.int8, device=A.device)
    if exp is None:
        exp = torch.empty(atb_bfp16_exp_bytes(M, K), dtype=torch.uint8, device=A.device)
    _check(load_library().atb_quantize_bfp16(_dev_ptr(A), M, K, A.stride(0) if M > 1 else max(K, A.stride(0)),
                                              _dev_ptr(mant), _dev_ptr(exp), _stream_ptr(stream)))
    return mant, exp


def atb_gemm(M, N, K, T_MA, T_MC, T_K, T_N, A_mant, A_exp, B, C=None, ldb=None, ldc=None, stream=None):
    """``C[M][N] = dequant(A) @ B``; B, C are bf16 CUDA tensors (row-major).  Returns C."""
    import torch
    if C is None:
        C = torch.empty((M, N), dtype=torch.bfloat16, device=B.device)
    if ldb is None:
        ldb = B.stride(0) if not isinstance(B, int) else N
    if ldc is None:
        ldc = C.stride(0) if not isinstance(C, int) else N
    _check(load_library().atb_gemm(M, N, K, T_MA, T_MC, T_K, T_N, _dev_ptr(A_mant), _dev_ptr(A_exp),
                                   _dev_ptr(B), ldb, _dev_ptr(C), ldc, _stream_ptr(stream)))
    return C


def atb_gemm_splitk_workspace_bytes(M: int, N: int, T_MC: int, splits: int) -> int:
    return int(load_library().atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits))


def atb_select_splits(M: int, N: int, K: int, T_MC: int, T_K: int, T_N: int) -> int:
    return int(load_library().atb_select_splits(M, N, K, T_MC, T_K, T_N))


def atb_gemm_splitk(M, N, K, T_MA, T_MC, T_K, T_N, A_mant, A_exp, B, splits, workspace=None, C=None, ldb=None,
                    ldc=None, stream=None):
    """Split-K ``C[M][N] = dequant(A) @ B``; ``workspace`` is a float32 CUDA tensor (allocated if None)."""
    import torch
    if C is None:
        C = torch.empty((M, N), dtype=torch.bfloat16, device=B.device)
    if workspace is None:
        workspace = torch.empty(atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits) // 4, dtype=torch.float32,
                                device=B.device)
    if ldb is None:
        ldb = B.stride(0)
    if ldc is None:
        ldc = C.stride(0)
    _check(load_library().atb_gemm_splitk(M, N, K, T_MA, T_MC, T_K, T_N, _dev_ptr(A_mant), _dev_ptr(A_exp), _dev_ptr(B),
                                          ldb, _dev_ptr(C), ldc, splits, _dev_ptr(workspace),
                                          workspace.numel() * workspace.element_size(), _stream_ptr(stream)))
    return C


def atb_gemm_bfp16_out(M, N, K, T_MA, T_MC, T_K, T_N, A_mant, A_exp, B, C_mant=None, C_exp=None, ldb=None, stream=None):
    """``C = dequant(A) @ B`` written as BFP16 planes (quantising epilogue).  Returns ``(C_mant, C_exp)``:
    an int8 ``[M, N]`` tensor and the exponent plane, both usable as the A operand of the next GEMM."""
    import torch
    if C_mant is None:
        C_mant = torch.empty((M, N), dtype=torch.int8, device=B.device)
    if C_exp is None:
        C_exp = torch.empty(atb_bfp16_exp_bytes(M, N), dtype=torch.uint8, device=B.device)
    if ldb is None:
        ldb = B.stride(0)
    _check(load_library().atb_gemm_bfp16_out(M, N, K, T_MA, T_MC, T_K, T_N, _dev_ptr(A_mant), _dev_ptr(A_exp), _dev_ptr(B),
                                             ldb, _dev_ptr(C_mant), _dev_ptr(C_exp), _stream_ptr(stream)))
    return C_mant, C_exp


def atb_gemm_config_tiled(config, M, N, K, T_MA, T_MC, T_K, T_N, A, A_exp, Bt_mant, Bt_exp, C=None, C_exp=None, stream=None):
    """The paper's precision configurations with the BFP16 operand on the B side (planes of B transposed),
    A streamed in slabs of ``T_MA`` rows; ``T_K, T_N`` = 64, 256 and ``T_MC`` = 256 (one SM) or 512 (a CTA pair
    that shares the converted B tile).

    ``config=1``: ``A`` is a bf16 ``[M, K]`` tensor (``A_exp=None``); returns bf16 ``C``.
    ``config=2``: ``A`` / ``A_exp`` are BFP16 planes; returns ``(C_mant, C_exp)``."""
    import torch
    dev = Bt_mant.device
    if config == 1:
        if C is None:
            C = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        _check(load_library().atb_gemm_config_tiled(1, M, N, K, T_MA, T_MC, T_K, T_N, _dev_ptr(A), None, A.stride(0),
                                                    _dev_ptr(Bt_mant), _dev_ptr(Bt_exp), _dev_ptr(C), None, C.stride(0),
                                                    _stream_ptr(stream)))
        return C
    if C is None:
        C = torch.empty((M, N), dtype=torch.int8, device=dev)
    if C_exp is None:
        C_exp = torch.empty(atb_bfp16_exp_bytes(M, N), dtype=torch.uint8, device=dev)
    _check(load_library().atb_gemm_config_tiled(config, M, N, K, T_MA, T_MC, T_K, T_N, _dev_ptr(A),
                                                _dev_ptr(A_exp) if A_exp is not None else None, K, _dev_ptr(Bt_mant),
                                                _dev_ptr(Bt_exp), _dev_ptr(C), _dev_ptr(C_exp), N, _stream_ptr(stream)))
    return C, C_exp


def atb_gemm_config(config, M, N, K, A, A_exp, Bt_mant, Bt_exp, C=None, C_exp=None, stream=None):
    """``atb_gemm_config_tiled`` with 128-row slabs, on a CTA pair where M > 256; goes through the C entry of the
    same name."""
    import torch
    dev = Bt_mant.device
    if config == 1:
        if C is None:
            C = torch.empty((M, N), dtype=torch.bfloat16, device=dev)
        _check(load_library().atb_gemm_config(1, M, N, K, _dev_ptr(A), None, A.stride(0), _dev_ptr(Bt_mant), _dev_ptr(Bt_exp),
                                              _dev_ptr(C), None, C.stride(0), _stream_ptr(stream)))
        return C
    if C is None:
        C = torch.empty((M, N), dtype=torch.int8, device=dev)
    if C_exp is None:
        C_exp = torch.empty(atb_bfp16_exp_bytes(M, N), dtype=torch.uint8, device=dev)
    _check(load_library().atb_gemm_config(config, M, N, K, _dev_ptr(A), _dev_ptr(A_exp) if A_exp is not None else None, K,
                                          _dev_ptr(Bt_mant), _dev_ptr(Bt_exp), _dev_ptr(C), _dev_ptr(C_exp), N,
                                          _stream_ptr(stream)))
    return C, C_exp


NOALLOC_SCRATCH_BYTES = 64 * 1024 * 1024


def atb_gemm_splitk_noalloc(M, N, K, T_MA, T_MC, T_K, T_N, A_mant, A_exp, B, splits, C, ldb=None, ldc=None, stream=None):
    """Split-K GEMM whose partial sums live in the library's built-in 64 MiB device array.

    For callers that may not allocate: the binding allocates nothing either, so ``C`` (bf16 CUDA tensor)
    has to be passed in.  Raises ``AtbError`` (ATB_ERR_BUFFER_TOO_SMALL) when
    ``atb_gemm_splitk_workspace_bytes(M, N, T_MC, splits)`` exceeds ``NOALLOC_SCRATCH_BYTES``.
    Calls that may overlap on the GPU must be ordered by the caller: they share the array."""
    if ldb is None:
        ldb = B.stride(0)
    if ldc is None:
        ldc = C.stride(0)
    _check(load_library().atb_gemm_splitk_noalloc(M, N, K, T_MA, T_MC, T_K, T_N, _dev_ptr(A_mant), _dev_ptr(A_exp),
                                                  _dev_ptr(B), ldb, _dev_ptr(C), ldc, splits, _stream_ptr(stream)))
    return C


def atb_device_status(stream=None):
    """Synchronises ``stream`` and raises ``AtbError`` if a kernel gave up a bounded wait."""
    _check(load_library().atb_device_status(_stream_ptr(stream)))


# ------------------------------------------------------------------ host model
def atb_hw_params_b200() -> atb_hw_params_t:
    hw = atb_hw_params_t()
    load_library().atb_hw_params_b200(ctypes.byref(hw))
    return hw


def atb_hw_params_xdna2(precision_config: int) -> atb_hw_params_t:
    hw = atb_hw_params_t()
    load_library().atb_hw_params_xdna2(ctypes.byref(hw), precision_config)
    return hw


def atb_score_tiling(hw: atb_hw_params_t, K: int, tiling) -> atb_tiling_score_t:
    out = atb_tiling_score_t()
    _check(load_library().atb_score_tiling(ctypes.byref(hw), K, atb_tiling_t(*tiling), ctypes.byref(out)))
    return out


def atb_select_tiling(M: int, N: int, K: int, hw: atb_hw_params_t | None = None, max_scores: int = 128):
    """Returns ``(best: Tiling, scores: list[atb_tiling_score_t])`` - scores best first."""
    best = atb_tiling_t()
    scores = (atb_tiling_score_t * max_scores)()
    n = ctypes.c_int(max_scores)
    _check(load_library().atb_select_tiling(M, N, K, ctypes.byref(hw) if hw is not None else None,
                                            ctypes.byref(best), scores, ctypes.byref(n)))
    return Tiling(best.T_MA, best.T_MC, best.T_K, best.T_N), [scores[i] for i in range(n.value)]


# ------------------------------------------------------------------ layout helpers (no arithmetic)
def exp_plane_to_logical(exp_plane, M: int, K: int):
    """Device exponent plane ``[ceil(K/64)][roundup(M,32)][8]`` -> logical ``[M][K/8]`` (numpy)."""
    import numpy as np
    e = np.asarray(exp_plane, dtype=np.uint8).reshape(-1)
    panels, m_pad = -(-K // 64), -(-M // 32) * 32
    e = e.reshape(panels, m_pad, 8).transpose(1, 0, 2).reshape(m_pad, panels * 8)
    return np.ascontiguousarray(e[:M, :K // 8])


def logical_to_exp_plane(exp_logical, M: int, K: int):
    """Logical ``[M][K/8]`` exponents -> flat device plane (numpy uint8, padding zero)."""
    import numpy as np
    panels, m_pad = -(-K // 64), -(-M // 32) * 32
    full = np.zeros((m_pad, panels * 8), np.uint8)
    full[:M, :K // 8] = np.asarray(exp_logical, dtype=np.uint8)
    return np.ascontiguousarray(full.reshape(m_pad, panels, 8).transpose(1, 0, 2)).reshape(-1)

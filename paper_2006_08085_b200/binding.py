"""ctypes binding of libdetag.so: the functions of include/detag.h under the same names.

Argument marshalling only.  Device buffers are ``torch`` CUDA tensors (or raw integer
addresses); streams are ``torch.cuda.Stream`` objects, raw handles or None.  Every function
raises ``DetagError`` on a negative return code.  There is no fallback: if the library has
not been built, or a call needs a GPU that is not there, the call fails.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdetag.so")

DETAG_OK = 0
DETAG_ERR_ARG = -1
DETAG_ERR_CSR = -2
DETAG_ERR_NOT_STOCHASTIC = -3
DETAG_ERR_NOT_SYMMETRIC = -4
DETAG_ERR_UNSUPPORTED = -5
DETAG_ERR_UNBOUND = -6
DETAG_ERR_CUDA = -7
DETAG_ERR_TIMEOUT = -8
DETAG_ERR_SPECTRUM = -9

DETAG_VARIANT_AUTO = 0
DETAG_VARIANT_CSR = 1
DETAG_VARIANT_DENSE = 2
DETAG_VARIANT_RING = 3
DETAG_VARIANT_TORUS = 4

DETAG_GRADIENT_AT_NEW_MODEL = 0
DETAG_GRADIENT_AT_PHASE_START = 1

DETAG_ALGORITHM_DETAG = 0
DETAG_ALGORITHM_DPSGD = 1

DETAG_GRADIENT_SYNTHETIC = 0
DETAG_GRADIENT_EXTERNAL = 1

_ERR_NAMES = {
    -1: "DETAG_ERR_ARG", -2: "DETAG_ERR_CSR", -3: "DETAG_ERR_NOT_STOCHASTIC", -4: "DETAG_ERR_NOT_SYMMETRIC",
    -5: "DETAG_ERR_UNSUPPORTED", -6: "DETAG_ERR_UNBOUND", -7: "DETAG_ERR_CUDA", -8: "DETAG_ERR_TIMEOUT",
    -9: "DETAG_ERR_SPECTRUM",
}

# every symbol include/detag.h declares: name -> (restype, argtypes)
_P = ctypes.c_void_p
_I32P = ctypes.POINTER(ctypes.c_int32)
_F64P = ctypes.POINTER(ctypes.c_double)
SIGNATURES = {
    "detag_spectral": (ctypes.c_int, [ctypes.c_int, _I32P, _I32P, _F64P, _F64P, _F64P, _F64P, _F64P]),
    "detag_create": (ctypes.c_int, [ctypes.POINTER(_P), ctypes.c_int, ctypes.c_int64, _I32P, _I32P, _F64P,
                                    ctypes.c_int, ctypes.c_double, ctypes.c_double]),
    "detag_workspace_bytes": (ctypes.c_int, [_P, ctypes.POINTER(ctypes.c_size_t)]),
    "detag_bind": (ctypes.c_int, [_P, ctypes.c_int64, _P, _P, _P, _P, _P, _P, ctypes.c_size_t]),
    "detag_observe_gossiped_tracker": (ctypes.c_int, [_P, _P]),
    "detag_set_noise": (ctypes.c_int, [_P, ctypes.c_double, ctypes.c_uint64, ctypes.c_int64]),
    "detag_set_variant": (ctypes.c_int, [_P, ctypes.c_int]),
    "detag_get_variant": (ctypes.c_int, [_P, ctypes.POINTER(ctypes.c_int)]),
    "detag_set_gradient_point": (ctypes.c_int, [_P, ctypes.c_int]),
    "detag_get_gradient_point": (ctypes.c_int, [_P, ctypes.POINTER(ctypes.c_int)]),
    "detag_set_algorithm": (ctypes.c_int, [_P, ctypes.c_int]),
    "detag_get_algorithm": (ctypes.c_int, [_P, ctypes.POINTER(ctypes.c_int)]),
    "detag_set_gradient_source": (ctypes.c_int, [_P, ctypes.c_int, _P]),
    "detag_debug_inject_stall": (ctypes.c_int, [_P, ctypes.c_int64, ctypes.c_uint32]),
    "detag_debug_expire_wait": (ctypes.c_int, [_P, ctypes.c_uint32, _P]),
    "detag_zero_chain_gradient": (ctypes.c_int, [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, _P, _P, ctypes.c_double,
                                                 ctypes.c_double, ctypes.c_double, ctypes.c_uint64, ctypes.c_int64, _P, _P]),
    "detag_phase_length": (ctypes.c_int, [ctypes.c_int, ctypes.c_double, ctypes.c_double, ctypes.c_double,
                                          ctypes.c_double, ctypes.POINTER(ctypes.c_int)]),
    "detag_init": (ctypes.c_int, [_P, _P]),
    "detag_step": (ctypes.c_int, [_P, _P]),
    "detag_step_many": (ctypes.c_int, [_P, ctypes.c_int, _P]),
    "detag_step_host": (ctypes.c_int, [_P, ctypes.c_int64, _P, _P, _P, _P, _P, _P, ctypes.c_size_t, _P]),
    "detag_host_staging_bytes": (ctypes.c_int, [_P, ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)]),
    "detag_consensus_error": (ctypes.c_int, [_P, _P, _F64P]),
    "detag_consensus_error_static": (ctypes.c_int, [ctypes.c_int, ctypes.c_int64, ctypes.c_int64, _P, _P, _F64P]),
    "detag_get_step": (ctypes.c_int, [_P, ctypes.POINTER(ctypes.c_int64)]),
    "detag_set_step": (ctypes.c_int, [_P, ctypes.c_int64]),
    "detag_status": (ctypes.c_int, [_P, _P]),
    "detag_last_error": (ctypes.c_char_p, [_P]),
    "detag_destroy": (ctypes.c_int, [_P]),
}

_lib: Optional[ctypes.CDLL] = None


class DetagError(RuntimeError):
    def __init__(self, code: int, where: str, text: str = ""):
        self.code = code
        super().__init__(f"{where}: {_ERR_NAMES.get(code, code)}" + (f" ({text})" if text else ""))


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built (no fallback path exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise FileNotFoundError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2006_08085_b200.build` "
                "(needs nvcc); the DeTAG step has no CPU fallback")
        handle = ctypes.CDLL(LIB_PATH)
        for name, (res, args) in SIGNATURES.items():
            fn = getattr(handle, name)
            fn.restype = res
            fn.argtypes = args
        _lib = handle
    return _lib


def _check(code: int, where: str, state=None) -> None:
    if code != DETAG_OK:
        text = ""
        if state is not None:
            text = (lib().detag_last_error(state) or b"").decode()
        raise DetagError(code, where, text)


def _dev_ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return int(t.data_ptr())


def _stream_handle(stream) -> Optional[int]:
    if stream is None:
        return None
    if isinstance(stream, int):
        return stream
    return int(stream.cuda_stream)


def _csr_args(row_ptr, col_idx, vals):
    rp = np.ascontiguousarray(row_ptr, dtype=np.int32)
    ci = np.ascontiguousarray(col_idx, dtype=np.int32)
    va = np.ascontiguousarray(vals, dtype=np.float64)
    return rp, ci, va, rp.ctypes.data_as(_I32P), ci.ctypes.data_as(_I32P), va.ctypes.data_as(_F64P)


def detag_spectral(n: int, row_ptr, col_idx, vals) -> Tuple[float, float, float, float]:
    """(lambda2, lambda_min, lambda, eta) of a symmetric gossip matrix given in CSR (host arrays)."""
    keep = _csr_args(row_ptr, col_idx, vals)
    out = [ctypes.c_double(float("nan")) for _ in range(4)]
    _check(lib().detag_spectral(n, keep[3], keep[4], keep[5], *[ctypes.byref(o) for o in out]), "detag_spectral")
    return tuple(o.value for o in out)


def detag_create(n: int, d: int, row_ptr, col_idx, vals, K: int, eta: float, alpha: float) -> ctypes.c_void_p:
    keep = _csr_args(row_ptr, col_idx, vals)
    handle = _P()
    _check(lib().detag_create(ctypes.byref(handle), n, d, keep[3], keep[4], keep[5], K, float(eta), float(alpha)),
           "detag_create")
    return handle


def detag_workspace_bytes(state) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().detag_workspace_bytes(state, ctypes.byref(out)), "detag_workspace_bytes", state)
    return int(out.value)


def detag_bind(state, ld: int, x, y, g, a, c, workspace, workspace_bytes: Optional[int] = None) -> None:
    if workspace_bytes is None:
        workspace_bytes = workspace.numel() * workspace.element_size()
    _check(lib().detag_bind(state, ld, _dev_ptr(x), _dev_ptr(y), _dev_ptr(g), _dev_ptr(a), _dev_ptr(c),
                            _dev_ptr(workspace), workspace_bytes), "detag_bind", state)


def detag_observe_gossiped_tracker(state, y_gossip) -> None:
    _check(lib().detag_observe_gossiped_tracker(state, _dev_ptr(y_gossip)), "detag_observe_gossiped_tracker", state)


def detag_set_noise(state, sigma: float, seed: int, coord_offset: int = 0) -> None:
    _check(lib().detag_set_noise(state, float(sigma), int(seed), int(coord_offset)), "detag_set_noise", state)


def detag_set_variant(state, variant: int) -> None:
    _check(lib().detag_set_variant(state, int(variant)), "detag_set_variant", state)


def detag_get_variant(state) -> int:
    out = ctypes.c_int(0)
    _check(lib().detag_get_variant(state, ctypes.byref(out)), "detag_get_variant", state)
    return int(out.value)


def detag_set_gradient_point(state, where: int) -> None:
    _check(lib().detag_set_gradient_point(state, int(where)), "detag_set_gradient_point", state)


def detag_get_gradient_point(state) -> int:
    out = ctypes.c_int(0)
    _check(lib().detag_get_gradient_point(state, ctypes.byref(out)), "detag_get_gradient_point", state)
    return int(out.value)


def detag_set_algorithm(state, algorithm: int) -> None:
    _check(lib().detag_set_algorithm(state, int(algorithm)), "detag_set_algorithm", state)


def detag_get_algorithm(state) -> int:
    out = ctypes.c_int(0)
    _check(lib().detag_get_algorithm(state, ctypes.byref(out)), "detag_get_algorithm", state)
    return int(out.value)


def detag_set_gradient_source(state, source: int, g_new=None) -> None:
    """g_new: device tensor [n][ld] float32 the caller writes the newest gradient into (external source only)."""
    _check(lib().detag_set_gradient_source(state, int(source), _dev_ptr(g_new)), "detag_set_gradient_source", state)


def detag_debug_inject_stall(state, after_tiles: int, poll_limit: int = 2048) -> None:
    _check(lib().detag_debug_inject_stall(state, int(after_tiles), int(poll_limit)), "detag_debug_inject_stall", state)


def detag_debug_expire_wait(state, polls: int, stream=None) -> None:
    _check(lib().detag_debug_expire_wait(state, int(polls), _stream_handle(stream)), "detag_debug_expire_wait", state)


def detag_zero_chain_gradient(n: int, d: int, ld: int, x, g_out, lam: float, gain: float, p: float, seed: int, t: int,
                              scratch, stream=None) -> None:
    """Bernoulli-progress gradient oracle of the zero-chain objective (proof of Theorem 1) into g_out; scratch is a
    device int32 tensor with n entries."""
    _check(lib().detag_zero_chain_gradient(int(n), int(d), int(ld), _dev_ptr(x), _dev_ptr(g_out), float(lam), float(gain),
                                           float(p), int(seed), int(t), _dev_ptr(scratch), _stream_handle(stream)),
           "detag_zero_chain_gradient")


def detag_phase_length(n: int, lam: float, varsigma0_sq: float = 0.0, T: float = 0.0, delta_L: float = 1.0) -> int:
    """Theorem 3's phase length (gossip rounds per phase), host only."""
    out = ctypes.c_int(0)
    _check(lib().detag_phase_length(int(n), float(lam), float(varsigma0_sq), float(T), float(delta_L),
                                    ctypes.byref(out)), "detag_phase_length")
    return int(out.value)


def detag_init(state, stream=None) -> None:
    _check(lib().detag_init(state, _stream_handle(stream)), "detag_init", state)


def detag_step(state, stream=None) -> None:
    _check(lib().detag_step(state, _stream_handle(stream)), "detag_step", state)


def detag_step_many(state, count: int, stream=None) -> None:
    """`count` iterations; where the variant allows it they run on chip in one launch (same bits as detag_step)."""
    _check(lib().detag_step_many(state, int(count), _stream_handle(stream)), "detag_step_many", state)


def detag_step_host(state, ld_host: int, x, y, g, a, c, staging, staging_bytes: int, stream=None) -> None:
    """x, y, g, a, c: host tensors (page-locked for overlap) or raw host addresses; staging: device memory."""
    _check(lib().detag_step_host(state, ld_host, _dev_ptr(x), _dev_ptr(y), _dev_ptr(g), _dev_ptr(a), _dev_ptr(c),
                                 _dev_ptr(staging), int(staging_bytes), _stream_handle(stream)),
           "detag_step_host", state)


def detag_host_staging_bytes(state, chunk_coords: int) -> int:
    out = ctypes.c_size_t(0)
    _check(lib().detag_host_staging_bytes(state, int(chunk_coords), ctypes.byref(out)), "detag_host_staging_bytes",
           state)
    return int(out.value)


def detag_consensus_error(state, stream=None) -> float:
    out = ctypes.c_double(float("nan"))
    _check(lib().detag_consensus_error(state, _stream_handle(stream), ctypes.byref(out)), "detag_consensus_error",
           state)
    return float(out.value)


def detag_consensus_error_static(n: int, d: int, ld: int, x, stream=None) -> float:
    """Consensus error of the device array x ([n][ld] float32) using only the library's built-in scratch
    array: for callers that cannot allocate device memory or pass a workspace.  d <= 33,554,432."""
    out = ctypes.c_double(float("nan"))
    _check(lib().detag_consensus_error_static(int(n), int(d), int(ld), _dev_ptr(x), _stream_handle(stream),
                                              ctypes.byref(out)), "detag_consensus_error_static")
    return float(out.value)


def detag_get_step(state) -> int:
    out = ctypes.c_int64(0)
    _check(lib().detag_get_step(state, ctypes.byref(out)), "detag_get_step", state)
    return int(out.value)


def detag_set_step(state, t: int) -> None:
    _check(lib().detag_set_step(state, int(t)), "detag_set_step", state)


def detag_status(state, stream=None) -> None:
    _check(lib().detag_status(state, _stream_handle(stream)), "detag_status", state)


def detag_last_error(state) -> str:
    return (lib().detag_last_error(state) or b"").decode()


def detag_destroy(state) -> None:
    _check(lib().detag_destroy(state), "detag_destroy")

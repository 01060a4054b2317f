"""ctypes binding of libtarflow.so: argument marshalling only.

Every function has the name and argument order of its C declaration in ``include/tarflow.h``.
Device buffers are torch CUDA tensors (torch is used for device memory and streams, nothing
else); the library is loaded from ``paper_2505_24791_b200/lib`` and a missing library is an
error -- there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

TF_OK, TF_MAXITER = 0, 1
TF_EINVAL, TF_ESIZE, TF_ENOMEM, TF_ECUDA, TF_ETIMEOUT, TF_ENONFINITE = -1, -2, -3, -4, -5, -6

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "lib", "libtarflow.so")


class TfConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("C", "H", "W", "patch", "n_blocks", "n_layers", "width", "n_heads",
                                         "mlp_ratio", "n_classes", "dtype", "max_batch")]


class TfMafConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("D", "hidden", "n_blocks", "dtype", "max_batch")]


class TfJacobiOpts(C.Structure):
    _fields_ = [("struct_bytes", C.c_int32), ("init_mode", C.c_int32), ("u0_dev", C.c_void_p),
                ("tau_block_host", C.c_void_p), ("fallback_sweeps", C.c_int32), ("reserved", C.c_int32),
                ("states_dev", C.c_void_p), ("ref_states_dev", C.c_void_p)]


class TarflowError(RuntimeError):
    def __init__(self, code, msg):
        super().__init__(f"libtarflow error {code}: {msg}")
        self.code = code


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -c 'import __graft_entry__ as g; "
                               "g.build()'` (there is no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        vp, i32, f32 = C.c_void_p, C.c_int32, C.c_float
        L.tf_load.argtypes = [C.POINTER(TfConfig), vp, C.c_size_t, C.POINTER(vp)]
        L.tf_free.argtypes = [vp]
        L.tf_free.restype = None
        L.tf_forward.argtypes = [vp, vp, vp, i32, vp, vp, vp]
        L.tf_inverse_sequential.argtypes = [vp, vp, vp, i32, vp, vp]
        L.tf_inverse_jacobi.argtypes = [vp, vp, vp, i32, vp, f32, i32, i32, vp, vp, vp, vp]
        L.tf_inverse_jacobi_ex.argtypes = [vp, vp, vp, i32, vp, f32, i32, C.POINTER(TfJacobiOpts), vp, vp, vp, vp]
        L.tf_block_times.argtypes = [vp, vp, i32]
        L.tf_trace_read_l2.argtypes = [vp, i32, i32, vp, i32]
        L.tf_maf_load.argtypes = [C.POINTER(TfMafConfig), vp, C.c_size_t, C.POINTER(vp)]
        L.tf_maf_forward.argtypes = [vp, vp, i32, vp, vp, vp]
        L.tf_maf_inverse_sequential.argtypes = [vp, vp, i32, vp, vp]
        L.tf_maf_inverse_jacobi.argtypes = [vp, vp, i32, f32, i32, i32, vp, vp, vp, vp]
        L.tf_inverse_jacobi_host.argtypes = [vp, vp, vp, i32, vp, f32, i32, i32, vp, vp, vp, vp]
        L.tf_jacobi_update.argtypes = [vp, vp, vp, vp, i32, i32, i32, i32, vp]
        L.tf_gemm_bf16.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
        L.tf_gemm_status.argtypes = [vp]
        L.tf_skinny_gemm_noalloc.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
        L.tf_profile_enable.argtypes = [vp, i32]
        L.tf_profile_read.argtypes = [vp, vp, vp, vp, vp, i32]
        L.tf_set_precision.argtypes = [vp, i32, f32, f32]
        L.tf_trace_enable.argtypes = [vp, i32]
        L.tf_trace_read.argtypes = [vp, vp, vp, vp, vp, i32]
        L.tf_selftest_wait_timeout.argtypes = [vp, i32, vp]
        L.tf_debug_check_guards.argtypes = [vp, vp]
        L.tf_debug_check_guards.restype = C.c_int64
        L.tf_launch_count.argtypes = [vp]
        L.tf_launch_count.restype = C.c_int64
        L.tf_device_bytes.argtypes = [vp]
        L.tf_device_bytes.restype = C.c_int64
        L.tf_last_error.restype = C.c_char_p
        _lib = L
    return _lib


def _check(code):
    if code < 0:
        raise TarflowError(code, lib().tf_last_error().decode())
    return code


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        import torch
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def make_config(cfg: dict, max_batch: int) -> TfConfig:
    return TfConfig(cfg["C"], cfg["H"], cfg["W"], cfg["patch"], cfg["n_blocks"], cfg["n_layers"], cfg["width"],
                    cfg["n_heads"], cfg["mlp_ratio"], cfg["n_classes"], cfg["dtype"], max_batch)


def tf_load(cfg: dict, blob: np.ndarray, max_batch: int):
    blob = np.ascontiguousarray(blob)
    out = C.c_void_p()
    c = make_config(cfg, max_batch)
    _check(lib().tf_load(C.byref(c), blob.ctypes.data_as(C.c_void_p), blob.nbytes, C.byref(out)))
    return out


def tf_free(m):
    lib().tf_free(m)


def tf_forward(m, x, labels, B, z, logdet, stream=None):
    return _check(lib().tf_forward(m, _ptr(x), _ptr(labels), B, _ptr(z), _ptr(logdet), _stream(stream)))


def tf_inverse_sequential(m, z, labels, B, x, stream=None):
    return _check(lib().tf_inverse_sequential(m, _ptr(z), _ptr(labels), B, _ptr(x), _stream(stream)))


def tf_inverse_jacobi(m, z, labels, B, policy, tau, max_iters, init_mode, x, iters_block=None, iters_sample=None,
                      stream=None):
    """policy: sequence of 0/1 per block; iters_block: numpy int32 [n_blocks] or None (host output)."""
    pol = np.ascontiguousarray(np.asarray(policy, dtype=np.uint8))
    ib = None if iters_block is None else iters_block.ctypes.data_as(C.c_void_p)
    return _check(lib().tf_inverse_jacobi(m, _ptr(z), _ptr(labels), B, pol.ctypes.data_as(C.c_void_p), tau, max_iters,
                                          init_mode, _ptr(x), ib, _ptr(iters_sample), _stream(stream)))


def tf_inverse_jacobi_ex(m, z, labels, B, policy, tau, max_iters, x, iters_block=None, iters_sample=None, stream=None,
                         init_mode=0, u0=None, tau_block=None, fallback_sweeps=0, states=None, ref_states=None):
    """Keyword arguments fill tf_jacobi_opts: u0 / states / ref_states are CUDA tensors [n_blocks,B,C,H,W], tau_block a
    sequence of floats per block."""
    pol = np.ascontiguousarray(np.asarray(policy, dtype=np.uint8))
    ib = None if iters_block is None else iters_block.ctypes.data_as(C.c_void_p)
    tb = None if tau_block is None else np.ascontiguousarray(np.asarray(tau_block, dtype=np.float32))
    o = TfJacobiOpts(C.sizeof(TfJacobiOpts), int(init_mode), None if u0 is None else u0.data_ptr(),
                     None if tb is None else tb.ctypes.data, int(fallback_sweeps), 0,
                     None if states is None else states.data_ptr(), None if ref_states is None else ref_states.data_ptr())
    return _check(lib().tf_inverse_jacobi_ex(m, _ptr(z), _ptr(labels), B, pol.ctypes.data_as(C.c_void_p), tau, max_iters,
                                             C.byref(o), _ptr(x), ib, _ptr(iters_sample), _stream(stream)))


def tf_block_times(m, n_blocks):
    """-> numpy float32 [n_blocks]: milliseconds of each block of the last inverse call (empty if none yet)."""
    ms = np.zeros(n_blocks, dtype=np.float32)
    k = _check(lib().tf_block_times(m, ms.ctypes.data_as(C.c_void_p), n_blocks))
    return ms[:k]


def tf_trace_read_l2(m, block, B, cap_sweeps=2048):
    """-> numpy float32 [sweeps, B]: ||u^t - ref||_2 per sweep and sample of a Jacobi block of the last _ex call."""
    buf = np.zeros((cap_sweeps, B), dtype=np.float32)
    n = _check(lib().tf_trace_read_l2(m, int(block), int(B), buf.ctypes.data_as(C.c_void_p), cap_sweeps))
    return buf[:min(n, cap_sweeps)]


def tf_inverse_jacobi_host(m, z_host, labels_host, B, policy, tau, max_iters, init_mode, x_host, iters_block=None,
                           iters_sample_host=None, stream=None):
    """z_host / x_host: CPU torch tensors (pinned for asynchronous copies) or numpy arrays."""
    pol = np.ascontiguousarray(np.asarray(policy, dtype=np.uint8))

    def hp(a):
        if a is None:
            return None
        return C.c_void_p(a.data_ptr()) if hasattr(a, "data_ptr") else a.ctypes.data_as(C.c_void_p)

    ib = None if iters_block is None else iters_block.ctypes.data_as(C.c_void_p)
    return _check(lib().tf_inverse_jacobi_host(m, hp(z_host), hp(labels_host), B, pol.ctypes.data_as(C.c_void_p), tau,
                                               max_iters, init_mode, hp(x_host), ib, hp(iters_sample_host),
                                               _stream(stream)))


def tf_maf_load(cfg: dict, blob: np.ndarray, max_batch: int):
    blob = np.ascontiguousarray(blob)
    out = C.c_void_p()
    c = TfMafConfig(cfg["D"], cfg["hidden"], cfg["n_blocks"], cfg["dtype"], max_batch)
    _check(lib().tf_maf_load(C.byref(c), blob.ctypes.data_as(C.c_void_p), blob.nbytes, C.byref(out)))
    return out


def tf_maf_forward(m, x, B, z, logdet, stream=None):
    return _check(lib().tf_maf_forward(m, _ptr(x), B, _ptr(z), _ptr(logdet), _stream(stream)))


def tf_maf_inverse_sequential(m, z, B, x, stream=None):
    return _check(lib().tf_maf_inverse_sequential(m, _ptr(z), B, _ptr(x), _stream(stream)))


def tf_maf_inverse_jacobi(m, z, B, tau, max_iters, init_mode, x, iters_block=None, iters_sample=None, stream=None):
    ib = None if iters_block is None else iters_block.ctypes.data_as(C.c_void_p)
    return _check(lib().tf_maf_inverse_jacobi(m, _ptr(z), B, tau, max_iters, init_mode, _ptr(x), ib, _ptr(iters_sample),
                                              _stream(stream)))


def tf_jacobi_update(o, v, u, maxdiff, B, L, D, reversed_, stream=None):
    return _check(lib().tf_jacobi_update(_ptr(o), _ptr(v), _ptr(u), _ptr(maxdiff), B, L, D, int(reversed_),
                                         _stream(stream)))


def tf_gemm_bf16(a, w, bias, c, M, N, K, stream=None):
    return _check(lib().tf_gemm_bf16(_ptr(a), _ptr(w), _ptr(bias), _ptr(c), M, N, K, _stream(stream)))


def tf_skinny_gemm_noalloc(a, w, bias, c, M, N, K, stream=None):
    return _check(lib().tf_skinny_gemm_noalloc(_ptr(a), _ptr(w), _ptr(bias), _ptr(c), M, N, K, _stream(stream)))


def tf_gemm_status(stream=None):
    return _check(lib().tf_gemm_status(_stream(stream)))


def tf_profile_enable(m, on):
    return _check(lib().tf_profile_enable(m, int(on)))


def tf_profile_read(m):
    """-> {kernel class: (milliseconds, launches, rows)} accumulated since tf_profile_enable."""
    cap = 64
    names = (C.c_char_p * cap)()
    ms = (C.c_double * cap)()
    n = (C.c_int64 * cap)()
    rows = (C.c_double * cap)()
    k = _check(lib().tf_profile_read(m, names, ms, n, rows, cap))
    return {names[i].decode(): (ms[i], n[i], rows[i]) for i in range(min(k, cap))}


def tf_set_precision(m, mode, switch_threshold=0.0, single_ok_tau=0.0):
    return _check(lib().tf_set_precision(m, int(mode), switch_threshold, single_ok_tau))


def tf_trace_enable(m, on):
    return _check(lib().tf_trace_enable(m, int(on)))


def tf_trace_read(m, cap=4096):
    """-> list of (block, sweep, active samples, max|u^t - u^(t-1)|) for the last inverse call."""
    blk, swp, act = ((C.c_int32 * cap)() for _ in range(3))
    md = (C.c_float * cap)()
    n = _check(lib().tf_trace_read(m, blk, swp, act, md, cap))
    return [(blk[i], swp[i], act[i], md[i]) for i in range(min(n, cap))]


def tf_selftest_wait_timeout(m, limit_us, stream=None):
    return _check(lib().tf_selftest_wait_timeout(m, int(limit_us), _stream(stream)))


def tf_debug_check_guards(m, stream=None):
    """-> number of overwritten guard words around the model's device buffers (0 = clean)."""
    n = lib().tf_debug_check_guards(m, _stream(stream))
    if n < 0:
        _check(int(n))
    return int(n)


def tf_launch_count(m):
    return lib().tf_launch_count(m)


def tf_device_bytes(m):
    return lib().tf_device_bytes(m)


def tf_last_error():
    return lib().tf_last_error().decode()

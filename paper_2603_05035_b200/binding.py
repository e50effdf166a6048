"""ctypes binding of ``libgelo.so`` -- argument marshalling only.

Every function here has the name and the arguments of the C entry point declared in
``include/gelo.h``; tensors are torch CUDA tensors whose ``data_ptr()`` is handed over.
All arithmetic of the path runs in the library's kernels.  A missing library is an
error: there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libgelo.so")
_lib = None

OK, ERR_INVALID, ERR_WORKSPACE, ERR_COND, ERR_TIMEOUT, ERR_CUDA, ERR_UNSUPPORTED = range(7)
ORTHOGONAL, NONORTHOGONAL = 0, 1
F32, BF16, F16 = 0, 1, 2
STREAM_G0, STREAM_G1, STREAM_SHIELD, STREAM_POWER = 0, 1, 2, 3

__all__ = [
    "OK", "ERR_INVALID", "ERR_WORKSPACE", "ERR_COND", "ERR_TIMEOUT", "ERR_CUDA", "ERR_UNSUPPORTED",
    "ORTHOGONAL", "NONORTHOGONAL", "F32", "BF16", "F16", "GeloError", "Context", "load_library", "library_path",
    "dtype_code", "EXPORTS",
]

_vp, _i, _u32, _u64, _f, _sz = (ctypes.c_void_p, ctypes.c_int, ctypes.c_uint32, ctypes.c_uint64,
                                ctypes.c_float, ctypes.c_size_t)

# name -> (restype, argtypes); mirrors include/gelo.h
EXPORTS = {
    "gelo_create": (_i, [ctypes.POINTER(_vp), _i]),
    "gelo_destroy": (_i, [_vp]),
    "gelo_workspace_bytes": (_sz, [_i, _i, _i, _i, _i]),
    "gelo_set_workspace": (_i, [_vp, _vp, _sz]),
    "gelo_set_nonorthogonal": (_i, [_vp, _f, _f, _i]),
    "gelo_mixing_ld": (_i, [_i]),
    "gelo_set_level3": (_i, [_vp, _i]),
    "gelo_last_status": (_i, [_vp, _vp]),
    "gelo_launch_count": (ctypes.c_longlong, [_vp, _i]),
    "gelo_status_string": (ctypes.c_char_p, [_i]),
    "gelo_philox_words": (_i, [_vp, _u64, _u32, _u32, _u64, _u64, _vp, _vp]),
    "gelo_sample_gaussian": (_i, [_vp, _i, _i, _i, _u64, _u32, _u32, _f, _vp, _vp]),
    "gelo_qr_orthogonal": (_i, [_vp, _i, _vp, _i, _vp, _vp, _vp]),
    "gelo_lu_inverse": (_i, [_vp, _i, _vp, _i, _vp, _vp]),
    "gelo_cond_estimate": (_i, [_vp, _i, _vp, _vp, _i, _vp, _vp]),
    "gelo_update_f32": (_i, [_vp, _i, _i, _i, _vp, _i, _vp, _i, _vp, _i, _vp]),
    "gelo_sample_mixing": (_i, [_vp, _i, _i, _u64, _i, _vp, _vp, _i, _vp, _vp]),
    "gelo_shield_rows": (_i, [_vp, _vp, _i, _i, _i, _f, _u64, _i, _vp, _vp]),
    "gelo_shield_rows_static": (_i, [_vp, _vp, _i, _i, _i, _f, _u64, _i, _vp, _vp]),
    "gelo_shield_rows_t": (_i, [_vp, _vp, _i, _i, _i, _f, _u64, _i, _i, _vp, _vp]),
    "gelo_set_shield_student_t": (_i, [_vp, _i]),
    "gelo_mix": (_i, [_vp, _vp, _i, _vp, _vp, _i, _i, _i, _i, _vp, _vp]),
    "gelo_project": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _vp, _vp]),
    "gelo_unmix": (_i, [_vp, _vp, _i, _vp, _i, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "gelo_quantize_e4m3": (_i, [_vp, _vp, _i, _i, _i, _vp, _vp, _vp]),
    "gelo_project_e4m3": (_i, [_vp, _vp, _vp, _vp, _vp, _i, _i, _i, _vp, _vp]),
    "gelo_qkv_offload": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _u64, _f, _i, _vp, _vp, _vp, _vp]),
    "gelo_project_unmix": (_i, [_vp, _vp, _vp, _vp, _i, _i, _i, _i, _i, _i, _vp, _vp, _vp, _vp]),
    "gelo_set_small_batch_fusion": (_i, [_vp, _i]),
    "gelo_qkv_offload_batch": (_i, [_vp, _i, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _f, _i, _vp, _vp, _vp, _vp]),
    "gelo_qkv_offload_batch_host": (_i, [_vp, _i, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _f, _i, _vp, _vp, _vp, _vp]),
    "gelo_blockdiag_workspace_bytes": (ctypes.c_size_t, [_i, _i, _i, _i, _i, _i, _i]),
    "gelo_qkv_offload_blockdiag_batch": (_i, [_vp, _i, _vp, _vp, _i, _i, _i, _i, _i, _vp, _f, _i, _vp, _vp, _vp, _vp]),
    "gelo_qkv_offload_batch_host_async": (_i, [_vp, _i, _vp, _vp, _i, _i, _i, _i, _vp, _vp, _f, _i, _vp, _vp, _vp, _vp]),
    "gelo_set_lanes": (_i, [_vp, _i]),
    "gelo_set_lane_share": (_i, [_vp, _i]),
    "gelo_set_wait_limit_ns": (_i, [_vp, ctypes.c_ulonglong]),
    "gelo_batch_workspace_bytes": (_sz, [_i, _i, _i, _i, _i, _i]),
    "gelo_profile_start": (_i, [_vp]),
    "gelo_profile_stop": (_i, [_vp, _vp, _vp]),
    "gelo_qkv_offload_host": (_i, [_vp, _vp, _vp, _i, _i, _i, _i, _i, _u64, _f, _i, _vp, _vp, _vp, _vp]),
}


class GeloError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        try:
            msg = load_library().gelo_status_string(status).decode()
        except Exception:  # pragma: no cover
            msg = "?"
        super().__init__(f"{where}: status {status} ({msg})")


def library_path() -> str:
    return _LIB_PATH


def load_library():
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(
                f"{_LIB_PATH} is missing: build it with `python -m paper_2603_05035_b200.build`")
        lib = ctypes.CDLL(_LIB_PATH)
        for name, (res, args) in EXPORTS.items():
            fn = getattr(lib, name)
            fn.restype = res
            fn.argtypes = args
        _lib = lib
    return _lib


def dtype_code(dtype) -> int:
    if dtype in (F32, "f32", torch.float32):
        return F32
    if dtype in (BF16, "bf16", torch.bfloat16):
        return BF16
    if dtype in ("f16", torch.float16) or (dtype == F16 and not isinstance(dtype, (str, torch.dtype))):
        return F16
    raise ValueError(f"unsupported dtype {dtype!r}")


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Context:
    """Owns a ``gelo_ctx`` and the torch tensor that serves as its workspace."""

    def __init__(self, device: int = 0):
        self._lib = load_library()
        self.device = int(device)
        h = _vp()
        self._check(self._lib.gelo_create(ctypes.byref(h), self.device), "gelo_create")
        self._h = h
        self._ws = None

    def close(self):
        if getattr(self, "_h", None):
            self._lib.gelo_destroy(self._h)
            self._h = None

    def __del__(self):  # pragma: no cover
        try:
            self.close()
        except Exception:
            pass

    def _check(self, status: int, where: str):
        if status != OK:
            raise GeloError(status, where)

    # ---- context -----------------------------------------------------------------
    def workspace_bytes(self, n, k, d, p, dtype) -> int:
        return int(self._lib.gelo_workspace_bytes(n, k, d, p, dtype_code(dtype)))

    def set_workspace(self, tensor_or_none):
        if tensor_or_none is None:
            self._check(self._lib.gelo_set_workspace(self._h, None, 0), "gelo_set_workspace")
            self._ws = None
            return
        t = tensor_or_none
        self._check(self._lib.gelo_set_workspace(self._h, t.data_ptr(), t.numel() * t.element_size()),
                    "gelo_set_workspace")
        self._ws = t

    def ensure_workspace(self, n, k, d, p, dtype):
        """Allocates (with torch) a workspace large enough for these sizes, if the current one is not."""
        need = self.workspace_bytes(n, k, d, p, dtype)
        if need == 0:
            raise ValueError("invalid sizes")
        if self._ws is None or self._ws.numel() < need:
            self.set_workspace(torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}"))
        return need

    def set_lanes(self, lanes: int):
        self._check(self._lib.gelo_set_lanes(self._h, lanes), "gelo_set_lanes")
        self.lanes = int(lanes)

    def set_lane_share(self, share: int):
        self._check(self._lib.gelo_set_lane_share(self._h, share), "gelo_set_lane_share")

    def set_wait_limit_ns(self, ns: int):
        """Limit of the device-side barrier waits of the tensor-core kernels (0: give up at once)."""
        self._check(self._lib.gelo_set_wait_limit_ns(self._h, int(ns)), "gelo_set_wait_limit_ns")

    def ensure_batch_workspace(self, n, k, d, p, dtype, lanes=None):
        """Workspace for the batched entry points with `lanes` concurrent sampling lanes."""
        lanes = int(lanes if lanes is not None else getattr(self, "lanes", 4))
        need = int(self._lib.gelo_batch_workspace_bytes(n, k, d, p, dtype_code(dtype), lanes))
        if need == 0:
            raise ValueError("invalid sizes")
        if self._ws is None or self._ws.numel() < need:
            self.set_workspace(torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}"))
        return need

    PROFILE_CLASSES = ("rank_update", "vtc", "gemm_tc", "qr_panel", "lu_panel")
    PROFILE_UNITS = ("bytes", "bytes", "flops", "flops", "flops")

    def profile_start(self):
        self._check(self._lib.gelo_profile_start(self._h), "gelo_profile_start")

    def profile_stop(self, stream=None):
        """{class: {"launches", "ms", "work", "unit"}} for the launches since profile_start."""
        out = (ctypes.c_double * 15)()
        self._check(self._lib.gelo_profile_stop(self._h, _stream(stream), ctypes.cast(out, ctypes.c_void_p)),
                    "gelo_profile_stop")
        return {name: {"launches": int(out[3 * i]), "ms": out[3 * i + 1], "work": out[3 * i + 2],
                       "unit": self.PROFILE_UNITS[i]} for i, name in enumerate(self.PROFILE_CLASSES)}

    def set_nonorthogonal(self, gamma=0.5, cond_bound=100.0, max_attempts=8):
        self._check(self._lib.gelo_set_nonorthogonal(self._h, gamma, cond_bound, max_attempts),
                    "gelo_set_nonorthogonal")

    def set_level3(self, mode: int):
        self._check(self._lib.gelo_set_level3(self._h, mode), "gelo_set_level3")

    def mixing_ld(self, m) -> int:
        return int(self._lib.gelo_mixing_ld(m))

    def last_status(self, stream=None) -> int:
        return int(self._lib.gelo_last_status(self._h, _stream(stream)))

    def launch_count(self, reset=False) -> int:
        return int(self._lib.gelo_launch_count(self._h, 1 if reset else 0))

    # ---- sampling -------------------------------------------------------------------
    def philox_words(self, seed, stream_id, attempt, first, count, out, stream=None):
        self._check(self._lib.gelo_philox_words(self._h, seed, stream_id, attempt, first, count, _ptr(out),
                                                _stream(stream)), "gelo_philox_words")

    def sample_gaussian(self, rows, cols, ld, seed, stream_id, attempt, scale, out, stream=None):
        self._check(self._lib.gelo_sample_gaussian(self._h, rows, cols, ld, seed, stream_id, attempt, scale,
                                                   _ptr(out), _stream(stream)), "gelo_sample_gaussian")

    def qr_orthogonal(self, m, G, ld, Q, Qt=None, stream=None):
        self._check(self._lib.gelo_qr_orthogonal(self._h, m, _ptr(G), ld, _ptr(Q), _ptr(Qt), _stream(stream)),
                    "gelo_qr_orthogonal")

    def lu_inverse(self, m, A, ld, Ainv, stream=None):
        self._check(self._lib.gelo_lu_inverse(self._h, m, _ptr(A), ld, _ptr(Ainv), _stream(stream)),
                    "gelo_lu_inverse")

    def cond_estimate(self, m, A, Ainv, ld, cond, stream=None):
        self._check(self._lib.gelo_cond_estimate(self._h, m, _ptr(A), _ptr(Ainv), ld, _ptr(cond),
                                                 _stream(stream)), "gelo_cond_estimate")

    def update_f32(self, M, N, K, A, lda, B, ldb, C, ldc, stream=None):
        self._check(self._lib.gelo_update_f32(self._h, M, N, K, _ptr(A), lda, _ptr(B), ldb, _ptr(C), ldc,
                                              _stream(stream)), "gelo_update_f32")

    def sample_mixing(self, m, kind, seed, dtype, A, Ainv, lda, cond=None, stream=None):
        self._check(self._lib.gelo_sample_mixing(self._h, m, kind, seed, dtype_code(dtype), _ptr(A), _ptr(Ainv),
                                                 lda, _ptr(cond), _stream(stream)), "gelo_sample_mixing")

    # ---- shields and products ----------------------------------------------------------
    def shield_rows(self, H, n, d, k, scale, seed, dtype, S, stream=None):
        self._check(self._lib.gelo_shield_rows(self._h, _ptr(H), n, d, k, scale, seed, dtype_code(dtype),
                                               _ptr(S), _stream(stream)), "gelo_shield_rows")

    def shield_rows_t(self, H, n, d, k, scale, seed, nu, dtype, S, stream=None):
        """Student-t shield rows with nu degrees of freedom (standardised to unit variance)."""
        self._check(self._lib.gelo_shield_rows_t(self._h, _ptr(H), n, d, k, scale, seed, nu, dtype_code(dtype),
                                                 _ptr(S), _stream(stream)), "gelo_shield_rows_t")

    def set_shield_student_t(self, nu: int):
        """Shield kind of the whole-call entry points: 0 Gaussian, else Student-t with nu degrees of freedom."""
        self._check(self._lib.gelo_set_shield_student_t(self._h, nu), "gelo_set_shield_student_t")

    def shield_rows_static(self, H, n, d, k, scale, seed, dtype, S, stream=None):
        """Shield rows for callers that cannot allocate: scratch lives inside the library (n <= 65536)."""
        self._check(self._lib.gelo_shield_rows_static(self._h, _ptr(H), n, d, k, scale, seed, dtype_code(dtype),
                                                      _ptr(S), _stream(stream)), "gelo_shield_rows_static")

    def mix(self, A, lda, H, S, n, k, d, dtype, U, stream=None):
        self._check(self._lib.gelo_mix(self._h, _ptr(A), lda, _ptr(H), _ptr(S), n, k, d, dtype_code(dtype),
                                       _ptr(U), _stream(stream)), "gelo_mix")

    def project(self, U, W, m, d, p, dtype, Yp, stream=None):
        self._check(self._lib.gelo_project(self._h, _ptr(U), _ptr(W), m, d, p, dtype_code(dtype), _ptr(Yp),
                                           _stream(stream)), "gelo_project")

    def quantize_e4m3(self, X, rows, cols, dtype, codes, scale, stream=None):
        """codes (uint8, rows x cols) and scale (two floats: the scale and a scratch slot) from X."""
        self._check(self._lib.gelo_quantize_e4m3(self._h, _ptr(X), rows, cols, dtype_code(dtype), _ptr(codes), _ptr(scale),
                                                 _stream(stream)), "gelo_quantize_e4m3")

    def project_e4m3(self, U8, u_scale, W8, w_scale, m, d, p, Yp, stream=None):
        """Yp (bf16) = u_scale * w_scale * (U8 @ W8) on E4M3 operands."""
        self._check(self._lib.gelo_project_e4m3(self._h, _ptr(U8), _ptr(u_scale), _ptr(W8), _ptr(w_scale), m, d, p, _ptr(Yp),
                                                _stream(stream)), "gelo_project_e4m3")

    def unmix(self, Ainv, lda, Yp, n, k, p, dtype, Q, K=None, V=None, stream=None):
        self._check(self._lib.gelo_unmix(self._h, _ptr(Ainv), lda, _ptr(Yp), n, k, p, dtype_code(dtype),
                                         _ptr(Q), _ptr(K), _ptr(V), _stream(stream)), "gelo_unmix")

    def project_unmix(self, U, W, Ainv, lda, n, k, d, p, dtype, Q, K=None, V=None, stream=None):
        """Projection and unmixing of a small batch (n + k <= 128) in one kernel."""
        self._check(self._lib.gelo_project_unmix(self._h, _ptr(U), _ptr(W), _ptr(Ainv), lda, n, k, d, p, dtype_code(dtype),
                                                 _ptr(Q), _ptr(K), _ptr(V), _stream(stream)), "gelo_project_unmix")

    def set_small_batch_fusion(self, on: bool):
        self._check(self._lib.gelo_set_small_batch_fusion(self._h, 1 if on else 0), "gelo_set_small_batch_fusion")

    def qkv_offload(self, H, W, n, k, d, p, kind, seed, shield_scale, dtype, Q, K=None, V=None, stream=None):
        self._check(self._lib.gelo_qkv_offload(self._h, _ptr(H), _ptr(W), n, k, d, p, kind, seed, shield_scale,
                                               dtype_code(dtype), _ptr(Q), _ptr(K), _ptr(V), _stream(stream)),
                    "gelo_qkv_offload")

    @staticmethod
    def _ptr_array(items, count):
        arr = (ctypes.c_void_p * count)()
        for i in range(count):
            arr[i] = _ptr(items[i]) if items is not None else None
        return arr

    def _batch(self, fn, name, H, W, n, k, d, p, kinds, seeds, shield_scale, dtype, Q, K, V, stream):
        calls = len(H)
        if not (len(W) == len(kinds) == len(seeds) == len(Q) == calls):
            raise ValueError("per-call lists must have one entry per call")
        kinds_a = (ctypes.c_int * calls)(*[int(x) for x in kinds])
        seeds_a = (ctypes.c_uint64 * calls)(*[int(x) for x in seeds])
        self._check(fn(self._h, calls, self._ptr_array(H, calls), self._ptr_array(W, calls), n, k, d, p, kinds_a,
                       seeds_a, shield_scale, dtype_code(dtype), self._ptr_array(Q, calls),
                       self._ptr_array(K, calls), self._ptr_array(V, calls), _stream(stream)), name)

    def qkv_offload_batch(self, H, W, n, k, d, p, kinds, seeds, shield_scale, dtype, Q, K=None, V=None, stream=None):
        """Lists with one entry per call; sampling of different calls runs on concurrent lanes."""
        self._batch(self._lib.gelo_qkv_offload_batch, "gelo_qkv_offload_batch", H, W, n, k, d, p, kinds, seeds,
                    shield_scale, dtype, Q, K, V, stream)

    def ensure_blockdiag_workspace(self, n, k, d, p, dtype, block, lanes=None):
        """Workspace for the block-diagonal variant."""
        lanes = int(lanes if lanes is not None else getattr(self, "lanes", 4))
        need = int(self._lib.gelo_blockdiag_workspace_bytes(n, k, d, p, dtype_code(dtype), block, lanes))
        if need == 0:
            raise ValueError("unsupported sizes for the block-diagonal variant")
        if self._ws is None or self._ws.numel() < need:
            self.set_workspace(torch.empty(need, dtype=torch.uint8, device=f"cuda:{self.device}"))
        return need

    def qkv_offload_blockdiag_batch(self, H, W, n, k, d, p, block, seeds, shield_scale, dtype, Q, K=None, V=None, stream=None):
        """Block-diagonal orthogonal mixing (structured variant); lists with one entry per call."""
        calls = len(H)
        if not (len(W) == len(seeds) == len(Q) == calls):
            raise ValueError("per-call lists must have one entry per call")
        seeds_a = (ctypes.c_uint64 * calls)(*[int(x) for x in seeds])
        self._check(self._lib.gelo_qkv_offload_blockdiag_batch(
            self._h, calls, self._ptr_array(H, calls), self._ptr_array(W, calls), n, k, d, p, block, seeds_a, shield_scale,
            dtype_code(dtype), self._ptr_array(Q, calls), self._ptr_array(K, calls), self._ptr_array(V, calls),
            _stream(stream)), "gelo_qkv_offload_blockdiag_batch")

    def qkv_offload_batch_host(self, H_host, W, n, k, d, p, kinds, seeds, shield_scale, dtype, Q_host, K_host=None,
                               V_host=None, stream=None):
        self._batch(self._lib.gelo_qkv_offload_batch_host, "gelo_qkv_offload_batch_host", H_host, W, n, k, d, p,
                    kinds, seeds, shield_scale, dtype, Q_host, K_host, V_host, stream)

    def qkv_offload_batch_host_async(self, H_host, W, n, k, d, p, kinds, seeds, shield_scale, dtype, Q_host, K_host=None,
                                     V_host=None, stream=None):
        """Enqueues the batch and returns; read the host results after synchronising the stream."""
        self._batch(self._lib.gelo_qkv_offload_batch_host_async, "gelo_qkv_offload_batch_host_async", H_host, W, n, k,
                    d, p, kinds, seeds, shield_scale, dtype, Q_host, K_host, V_host, stream)

    def qkv_offload_host(self, H_host, W, n, k, d, p, kind, seed, shield_scale, dtype, Q_host, K_host=None,
                         V_host=None, stream=None):
        self._check(self._lib.gelo_qkv_offload_host(self._h, _ptr(H_host), _ptr(W), n, k, d, p, kind, seed,
                                                    shield_scale, dtype_code(dtype), _ptr(Q_host), _ptr(K_host),
                                                    _ptr(V_host), _stream(stream)), "gelo_qkv_offload_host")

"""Thin ctypes binding of the C ABI declared in include/slim.h.

Argument marshalling only: every function checks dtypes/devices, takes raw device
pointers from torch tensors and the current CUDA stream, and calls the entry point
of the same name.  There is no fallback: if the CUDA library has not been built
the first call raises.
"""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

from .build import LIB_PATH

GROUP = 128
GEMV_MAX_M = 16

_lib = None


class SlimError(RuntimeError):
    def __init__(self, fn: str, status: int, text: str, cuda_error: int):
        super().__init__(f"{fn} failed: {text} (status {status}, cuda error {cuda_error})")
        self.status = status
        self.cuda_error = cuda_error


def lib():
    """Loads libslim_b200.so (built by paper_2405_14917_b200.build.build())."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"CUDA library not built: {LIB_PATH} is missing; run "
                               "`python -m paper_2405_14917_b200.build` (there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
        L.slim_version.restype = i
        L.slim_version.argtypes = []
        L.slim_status_string.restype = ctypes.c_char_p
        L.slim_status_string.argtypes = [i]
        L.slim_last_cuda_error.restype = i
        L.slim_last_cuda_error.argtypes = []
        sigs = {
            "slim_packed_bytes": [i, i, i, vp, ctypes.POINTER(sz)],
            "slim_workspace_bytes": [i, i, i, i, vp, ctypes.POINTER(sz)],
            "slim_workspace_init": [vp, sz, vp],
            "slim_workspace_status": [vp, vp],
            "slim_selftest_wait_timeout": [vp, sz, ctypes.c_uint, vp],
            "slim_pack_weights": [vp, vp, vp, i, i, i, vp],
            "slim_dequant": [vp, vp, vp, vp, vp, i, i, i, vp],
            "slim_mpq_gemv": [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp],
            "slim_mpq_gemm": [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, sz, vp],
            "slim_gemv_plan": [i, i, i, i, vp, vp],
            "slim_quantize_sqc": [vp, vp, vp, vp, vp, vp, i, i, i, ctypes.c_double, i, vp],
            "slim_mpq_gemm_static": [vp, vp, vp, vp, vp, vp, i, i, i, i, vp, vp],
            "slim_group_salience": [vp, vp, vp, i, i, i, vp],
            "slim_allocate_bits": [vp, i, i, i, vp],
            "slim_quantize_minmax": [vp, vp, vp, vp, vp, i, i, i, vp],
            "slim_quantize_minmax_sign1": [vp, vp, vp, vp, vp, i, i, i, vp],
            "slim_quantize_minmax_groups": [vp, vp, vp, vp, vp, i, i, i, vp, i, vp],
            "slim_gemv_set_bytes": [vp, i, i, ctypes.POINTER(sz), ctypes.POINTER(sz)],
            "slim_gemv_set_plan": [vp, i, i, vp, sz, vp, vp],
            "slim_mpq_gemv_set": [vp, vp, vp, sz, vp],
            "slim_dense_linear": [vp, vp, vp, i, i, i, vp],
            "slim_softmax_kl": [vp, vp, vp, i, i, vp],
            "slim_sba_workspace_bytes": [i, i, i, i, i, ctypes.POINTER(sz)],
            "slim_sba_search": [vp, vp, vp, i, i, i, i, i, i, vp, sz, vp, vp, vp, vp],
            "slim_gptq_workspace_bytes": [i, i, i, i, ctypes.POINTER(sz)],
            "slim_gptq_factor": [vp, i, i, ctypes.c_double, vp, vp, vp, sz, vp],
            "slim_gptq_quantize": [vp, vp, vp, ctypes.c_double, i, vp, vp, vp, vp, i, i, i, i, vp, sz, vp],
        }
        for name, args in sigs.items():
            fn = getattr(L, name)
            fn.restype = i
            fn.argtypes = args
        _lib = L
    return _lib


def _check(fn: str, status: int):
    if status != 0:
        L = lib()
        raise SlimError(fn, status, L.slim_status_string(status).decode(), L.slim_last_cuda_error())


def _bits(bits) -> np.ndarray:
    b = np.ascontiguousarray(np.asarray(bits), dtype=np.uint8)
    assert b.ndim == 1
    return b


def _bp(b: np.ndarray):
    return b.ctypes.data_as(ctypes.c_void_p)


def _dev(t: torch.Tensor, dtype, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == dtype and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA tensor of dtype {dtype}")
    return t.data_ptr()


def _stream(t: torch.Tensor) -> int:
    return torch.cuda.current_stream(t.device).cuda_stream


def version() -> int:
    return lib().slim_version()


def packed_bytes(N: int, K: int, bits, g: int = GROUP) -> int:
    b = _bits(bits)
    out = ctypes.c_size_t(0)
    _check("slim_packed_bytes", lib().slim_packed_bytes(N, K, g, _bp(b), ctypes.byref(out)))
    return out.value


def workspace_bytes(M: int, N: int, K: int, bits, g: int = GROUP) -> int:
    b = _bits(bits)
    out = ctypes.c_size_t(0)
    _check("slim_workspace_bytes", lib().slim_workspace_bytes(M, N, K, g, _bp(b), ctypes.byref(out)))
    return out.value


def gemv_plan(M: int, N: int, K: int, bits, g: int = GROUP) -> dict:
    """Launch plan of slim_mpq_gemv for this shape (host-only)."""
    b = _bits(bits)
    out = (ctypes.c_int * 6)()
    _check("slim_gemv_plan", lib().slim_gemv_plan(M, N, K, g, _bp(b), ctypes.cast(out, ctypes.c_void_p)))
    return dict(zip(("tiles_per_cta", "k_slices", "row_blocks", "smem_bytes", "n_tiles", "groups_per_chunk"), list(out)))


def workspace_init(workspace: torch.Tensor) -> None:
    p = _dev(workspace, torch.uint8, "workspace")
    _check("slim_workspace_init", lib().slim_workspace_init(p, workspace.numel(), _stream(workspace)))


def workspace_status(workspace: torch.Tensor) -> None:
    """Synchronises; raises SlimError(SLIM_ERR_TIMEOUT) if a kernel gave up a bounded wait."""
    p = _dev(workspace, torch.uint8, "workspace")
    _check("slim_workspace_status", lib().slim_workspace_status(p, _stream(workspace)))


def selftest_wait_timeout(workspace: torch.Tensor, limit_us: int = 1000) -> None:
    """Enqueues the kernel whose bounded wait runs out after limit_us microseconds (slim_selftest_wait_timeout)."""
    p = _dev(workspace, torch.uint8, "workspace")
    _check("slim_selftest_wait_timeout", lib().slim_selftest_wait_timeout(p, workspace.numel(), int(limit_us), _stream(workspace)))


def new_workspace(M: int, N: int, K: int, bits, device="cuda", g: int = GROUP) -> torch.Tensor:
    """Allocates (torch) and initialises a workspace large enough for this shape."""
    ws = torch.empty(workspace_bytes(M, N, K, bits, g), dtype=torch.uint8, device=device)
    workspace_init(ws)
    return ws


def pack_weights(codes: torch.Tensor, bits, packed: torch.Tensor | None = None, g: int = GROUP) -> torch.Tensor:
    b = _bits(bits)
    N, K = codes.shape
    if packed is None:
        packed = torch.empty(packed_bytes(N, K, b, g), dtype=torch.uint8, device=codes.device)
    _check("slim_pack_weights", lib().slim_pack_weights(_dev(codes, torch.uint8, "codes"), _bp(b),
                                                        _dev(packed, torch.uint8, "packed"), N, K, g, _stream(codes)))
    return packed


def dequant(packed: torch.Tensor, bits, scales: torch.Tensor, zeros: torch.Tensor, N: int, K: int,
            out: torch.Tensor | None = None, g: int = GROUP) -> torch.Tensor:
    b = _bits(bits)
    if out is None:
        out = torch.empty((N, K), dtype=torch.float16, device=packed.device)
    _check("slim_dequant", lib().slim_dequant(_dev(packed, torch.uint8, "packed"), _bp(b),
                                              _dev(scales, torch.float16, "scales"), _dev(zeros, torch.float16, "zeros"),
                                              _dev(out, torch.float16, "W"), N, K, g, _stream(packed)))
    return out


def _linear(fn_name: str, x, packed, bits, scales, zeros, N, workspace, out, g: int = GROUP):
    b = _bits(bits)
    M, K = x.shape
    if out is None:
        out = torch.empty((M, N), dtype=torch.float16, device=x.device)
    wp = _dev(workspace, torch.uint8, "workspace") if workspace is not None else None
    wb = workspace.numel() if workspace is not None else 0
    fn = getattr(lib(), fn_name)
    _check(fn_name, fn(_dev(x, torch.float16, "x"), _dev(packed, torch.uint8, "packed"), _bp(b),
                       _dev(scales, torch.float16, "scales"), _dev(zeros, torch.float16, "zeros"),
                       _dev(out, torch.float16, "y"), M, N, K, g, wp, wb, _stream(x)))
    return out


def mpq_gemv(x, packed, bits, scales, zeros, N: int, workspace, out=None, g: int = GROUP) -> torch.Tensor:
    """y = x W-hat^T for 1 <= M <= 16 (decode path)."""
    return _linear("slim_mpq_gemv", x, packed, bits, scales, zeros, N, workspace, out, g)


def mpq_gemm(x, packed, bits, scales, zeros, N: int, workspace, out=None, g: int = GROUP) -> torch.Tensor:
    """y = x W-hat^T for M > 16 (batched tensor-core path)."""
    return _linear("slim_mpq_gemm", x, packed, bits, scales, zeros, N, workspace, out, g)


def mpq_gemm_static(x, packed, bits, scales, zeros, N: int, out: torch.Tensor, status: torch.Tensor | None = None,
                    g: int = GROUP) -> torch.Tensor:
    """slim_mpq_gemm without a caller workspace: the library's built-in scratch array is used.

    For callers that may not allocate device memory, so `out` (fp16 [M][N]) and the optional
    `status` (one int32 word on the device) must be passed in; nothing is allocated here either.
    Calls on one device share the scratch: keep them on one stream.
    """
    b = _bits(bits)
    M, K = x.shape
    sp = _dev(status, torch.int32, "status") if status is not None else None
    _check("slim_mpq_gemm_static", lib().slim_mpq_gemm_static(
        _dev(x, torch.float16, "x"), _dev(packed, torch.uint8, "packed"), _bp(b), _dev(scales, torch.float16, "scales"),
        _dev(zeros, torch.float16, "zeros"), _dev(out, torch.float16, "y"), M, N, K, g, sp, _stream(x)))
    return out


def group_salience(W: torch.Tensor, act_norm: torch.Tensor, g: int = GROUP) -> torch.Tensor:
    N, K = W.shape
    out = torch.empty(K // g, dtype=torch.float64, device=W.device)
    _check("slim_group_salience", lib().slim_group_salience(_dev(W, torch.float16, "W"), _dev(act_norm, torch.float32, "act_norm"),
                                                            _dev(out, torch.float64, "salience"), N, K, g, _stream(W)))
    return out


def allocate_bits(salience, avg_bits: int, p: int = -1) -> np.ndarray:
    s = np.ascontiguousarray(np.asarray(salience), dtype=np.float64)
    out = np.zeros(s.shape[0], dtype=np.uint8)
    _check("slim_allocate_bits", lib().slim_allocate_bits(s.ctypes.data_as(ctypes.c_void_p), s.shape[0], avg_bits, p, _bp(out)))
    return out


def quantize_minmax(W: torch.Tensor, bits, one_bit: str = "minmax", g: int = GROUP):
    """Eq. 1 per (row, group); one_bit="sign_alpha" binarises the one-bit groups with Eq. 2 instead."""
    if one_bit not in ("minmax", "sign_alpha"):
        raise ValueError("one_bit must be 'minmax' or 'sign_alpha'")
    fn_name = "slim_quantize_minmax" if one_bit == "minmax" else "slim_quantize_minmax_sign1"
    b = _bits(bits)
    N, K = W.shape
    G = K // g
    codes = torch.empty((N, K), dtype=torch.uint8, device=W.device)
    scales = torch.empty((G, N), dtype=torch.float16, device=W.device)
    zeros = torch.empty((G, N), dtype=torch.float16, device=W.device)
    _check(fn_name, getattr(lib(), fn_name)(_dev(W, torch.float16, "W"), _bp(b), _dev(codes, torch.uint8, "codes"),
                                            _dev(scales, torch.float16, "scales"), _dev(zeros, torch.float16, "zeros"),
                                            N, K, g, _stream(W)))
    return codes, scales, zeros


def quantize_minmax_groups(W: torch.Tensor, bits, groups, codes: torch.Tensor, scales: torch.Tensor, zeros: torch.Tensor,
                           g: int = GROUP) -> None:
    """Re-quantises (Eq. 1) only the listed groups under `bits`, in place in codes / scales / zeros."""
    b = _bits(bits)
    gl = np.ascontiguousarray(np.asarray(groups), dtype=np.int32)
    N, K = W.shape
    _check("slim_quantize_minmax_groups", lib().slim_quantize_minmax_groups(
        _dev(W, torch.float16, "W"), _bp(b), _dev(codes, torch.uint8, "codes"), _dev(scales, torch.float16, "scales"),
        _dev(zeros, torch.float16, "zeros"), N, K, g, gl.ctypes.data, int(gl.size), _stream(W)))


def quantize_sqc(W: torch.Tensor, bits, lam: float = 0.1, n: int = 50, g: int = GROUP):
    """SQC line search (Algorithm 2) on the device.  Returns codes, scales, zeros, tau index."""
    b = _bits(bits)
    N, K = W.shape
    G = K // g
    codes = torch.empty((N, K), dtype=torch.uint8, device=W.device)
    scales = torch.empty((G, N), dtype=torch.float16, device=W.device)
    zeros = torch.empty((G, N), dtype=torch.float16, device=W.device)
    tau = torch.empty((G, N), dtype=torch.int32, device=W.device)
    _check("slim_quantize_sqc", lib().slim_quantize_sqc(_dev(W, torch.float16, "W"), _bp(b), _dev(codes, torch.uint8, "codes"),
                                                        _dev(scales, torch.float16, "scales"), _dev(zeros, torch.float16, "zeros"),
                                                        _dev(tau, torch.int32, "tau_index"), N, K, g, float(lam), int(n), _stream(W)))
    return codes, scales, zeros, tau


def dense_linear(x: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
    """y = x W^T in full precision (fp16 in, fp32 accumulate and out): the reference output of SBA."""
    M, K = x.shape
    N = W.shape[0]
    y = torch.empty((M, N), dtype=torch.float32, device=x.device)
    _check("slim_dense_linear", lib().slim_dense_linear(_dev(x, torch.float16, "x"), _dev(W, torch.float16, "W"),
                                                        _dev(y, torch.float32, "y"), M, N, K, _stream(x)))
    return y


def softmax_kl(y_ref: torch.Tensor, y_q: torch.Tensor) -> torch.Tensor:
    """KL divergence between softmax(y_ref[t]) and softmax(y_q[t]) per token t (fp64)."""
    M, N = y_ref.shape
    kl = torch.empty(M, dtype=torch.float64, device=y_ref.device)
    _check("slim_softmax_kl", lib().slim_softmax_kl(_dev(y_ref, torch.float32, "y_ref"), _dev(y_q, torch.float16, "y_q"),
                                                    _dev(kl, torch.float64, "kl"), M, N, _stream(y_ref)))
    return kl


def sba_workspace_bytes(M: int, N: int, K: int, avg_bits: int, g: int = GROUP) -> int:
    out = ctypes.c_size_t(0)
    _check("slim_sba_workspace_bytes", lib().slim_sba_workspace_bytes(M, N, K, g, avg_bits, ctypes.byref(out)))
    return out.value


def sba_search(W: torch.Tensor, x: torch.Tensor, act_norm: torch.Tensor, avg_bits: int, include_uniform: bool = True,
               workspace: torch.Tensor | None = None, g: int = GROUP):
    """Salience-Determined Bit Allocation search (func SBA of Algorithm 2) on the device.
    Returns (p_star, bits[G] (numpy), errors (numpy, one per candidate p))."""
    N, K = W.shape
    M = x.shape[0]
    G = K // g
    if workspace is None:
        workspace = torch.empty(sba_workspace_bytes(M, N, K, avg_bits, g), dtype=torch.uint8, device=W.device)
    p_star = ctypes.c_int(-1)
    bits = np.zeros(G, dtype=np.uint8)
    errors = np.zeros(G // 2 + 1 - (0 if include_uniform else 1), dtype=np.float64)
    _check("slim_sba_search", lib().slim_sba_search(_dev(W, torch.float16, "W"), _dev(x, torch.float16, "x"),
                                                    _dev(act_norm, torch.float32, "act_norm"), M, N, K, g, avg_bits,
                                                    1 if include_uniform else 0, _dev(workspace, torch.uint8, "workspace"),
                                                    workspace.numel(), ctypes.addressof(p_star), bits.ctypes.data,
                                                    errors.ctypes.data, _stream(W)))
    return p_star.value, bits, errors


def gptq_workspace_bytes(T: int, N: int, K: int, g: int = GROUP) -> int:
    out = ctypes.c_size_t(0)
    _check("slim_gptq_workspace_bytes", lib().slim_gptq_workspace_bytes(T, N, K, g, ctypes.byref(out)))
    return out.value


def gptq_factor(x: torch.Tensor, lam: float = 0.01, workspace: torch.Tensor | None = None):
    """Second step of Algorithm 1 on the device: U (fp64 [K][K], upper triangular) with
    U^T U = (H + lambda I)^-1 for H = x^T x / T, and the flags of the input channels that are zero in
    every token.  Returns (U, dead)."""
    T, K = x.shape
    if workspace is None:
        workspace = torch.empty(gptq_workspace_bytes(T, 0, K), dtype=torch.uint8, device=x.device)
    U = torch.empty(K, K, dtype=torch.float64, device=x.device)
    dead = torch.empty(K, dtype=torch.uint8, device=x.device)
    _check("slim_gptq_factor", lib().slim_gptq_factor(_dev(x, torch.float16, "x"), T, K, float(lam), U.data_ptr(), dead.data_ptr(),
                                                      _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(x)))
    return U, dead


def gptq_quantize(W: torch.Tensor, x: torch.Tensor, bits, lam: float = 0.01, quantizer: str = "sqc",
                  workspace: torch.Tensor | None = None, return_running: bool = False, g: int = GROUP):
    """Main loop of Algorithm 1 under a given bit map: group by group, quantise the running weights
    (SQC or Eq. 1) and push the group's error onto the columns still to come.  W fp16 [N][K], x fp16
    [T][K] calibration tokens.  Returns (codes uint8 [N][K], scales fp16 [G][N], zeros fp16 [G][N])
    and, if asked, the fp64 running weights after the last update."""
    if quantizer not in ("sqc", "minmax"):
        raise ValueError(quantizer)
    N, K = W.shape
    T = x.shape[0]
    b = _bits(bits)
    G = K // g
    if workspace is None:
        workspace = torch.empty(gptq_workspace_bytes(T, N, K, g), dtype=torch.uint8, device=W.device)
    codes = torch.empty(N, K, dtype=torch.uint8, device=W.device)
    scales = torch.empty(G, N, dtype=torch.float16, device=W.device)
    zeros = torch.empty(G, N, dtype=torch.float16, device=W.device)
    running = torch.empty(N, K, dtype=torch.float64, device=W.device) if return_running else None
    _check("slim_gptq_quantize", lib().slim_gptq_quantize(
        _dev(W, torch.float16, "W"), _dev(x, torch.float16, "x"), _bp(b), float(lam), 1 if quantizer == "sqc" else 0,
        codes.data_ptr(), scales.data_ptr(), zeros.data_ptr(), running.data_ptr() if return_running else None,
        N, K, T, g, _dev(workspace, torch.uint8, "workspace"), workspace.numel(), _stream(W)))
    return (codes, scales, zeros, running) if return_running else (codes, scales, zeros)


class _Layer(ctypes.Structure):
    """struct slim_layer"""
    _fields_ = [("x", ctypes.c_void_p), ("packed", ctypes.c_void_p), ("scales", ctypes.c_void_p), ("zeros", ctypes.c_void_p),
                ("y", ctypes.c_void_p), ("bits_host", ctypes.c_void_p), ("M", ctypes.c_int), ("N", ctypes.c_int), ("K", ctypes.c_int)]


class _SetInfo(ctypes.Structure):
    """struct slim_gemv_set_info"""
    _fields_ = [("n_layers", ctypes.c_int), ("grid", ctypes.c_int), ("n_slots", ctypes.c_int), ("slot_bytes", ctypes.c_int),
                ("token_tiles", ctypes.c_int), ("stage_tasks", ctypes.c_int), ("n_items", ctypes.c_int), ("max_bits", ctypes.c_int),
                ("max_tokens", ctypes.c_int), ("tiles_per_warp", ctypes.c_int), ("split", ctypes.c_int), ("n_counters", ctypes.c_int),
                ("resident_pairs", ctypes.c_int), ("resident_cluster", ctypes.c_int),
                ("plan_bytes", ctypes.c_size_t), ("workspace_bytes", ctypes.c_size_t), ("resident_smem", ctypes.c_size_t)]


class LayerSet:
    """Several independent decode-path layers run by one launch (slim_gemv_set_plan / slim_mpq_gemv_set).

    entries: sequence of (layer: QuantLinear, x: fp16 CUDA [M][K], y: fp16 CUDA [M][N]).  The plan
    and the workspace are torch tensors owned by this object; the tensors of the entries are kept
    alive with it."""

    def __init__(self, entries, g: int = GROUP):
        entries = list(entries)
        if not entries:
            raise ValueError("a layer set needs at least one layer")
        self._keep = entries
        self._bits = [_bits(L.bits) for (L, _, _) in entries]
        arr = (_Layer * len(entries))()
        for k, (L, x, y) in enumerate(entries):
            M = x.shape[0]
            if tuple(x.shape) != (M, L.K) or tuple(y.shape) != (M, L.N):
                raise ValueError(f"layer {k}: x must be [M][{L.K}] and y [M][{L.N}]")
            arr[k] = _Layer(_dev(x, torch.float16, "x"), _dev(L.packed, torch.uint8, "packed"), _dev(L.scales, torch.float16, "scales"),
                            _dev(L.zeros, torch.float16, "zeros"), _dev(y, torch.float16, "y"), self._bits[k].ctypes.data,
                            M, L.N, L.K)
        self._arr = arr
        device = entries[0][1].device
        pb, wb = ctypes.c_size_t(0), ctypes.c_size_t(0)
        _check("slim_gemv_set_bytes", lib().slim_gemv_set_bytes(ctypes.cast(arr, ctypes.c_void_p), len(entries), g,
                                                              ctypes.byref(pb), ctypes.byref(wb)))
        self.plan = torch.empty(pb.value, dtype=torch.uint8, device=device)
        self.workspace = torch.empty(max(wb.value, 256), dtype=torch.uint8, device=device)
        workspace_init(self.workspace)
        self._info = _SetInfo()
        _check("slim_gemv_set_plan", lib().slim_gemv_set_plan(ctypes.cast(arr, ctypes.c_void_p), len(entries), g, self.plan.data_ptr(),
                                                            self.plan.numel(), ctypes.addressof(self._info), _stream(self.plan)))

    @property
    def info(self) -> dict:
        return {name: getattr(self._info, name) for name, _ in _SetInfo._fields_}

    def run(self) -> None:
        """Enqueues the set on the current stream: y of every entry is overwritten."""
        _check("slim_mpq_gemv_set", lib().slim_mpq_gemv_set(ctypes.addressof(self._info), self.plan.data_ptr(), self.workspace.data_ptr(),
                                                          self.workspace.numel(), _stream(self.plan)))

    def check(self) -> None:
        workspace_status(self.workspace)


class QuantLinear:
    """One quantised layer resident on the device: packed codes, scales, zeros, bit map."""

    def __init__(self, packed, bits, scales, zeros, N: int, K: int, g: int = GROUP):
        self.packed, self.bits, self.scales, self.zeros, self.N, self.K, self.g = packed, _bits(bits), scales, zeros, N, K, g

    @classmethod
    def from_weight(cls, W: torch.Tensor, act_norm: torch.Tensor, avg_bits: int, p: int = -1, g: int = GROUP) -> "QuantLinear":
        """Salience -> bit allocation -> Eq. 1 quantizer -> packing, all on the device."""
        N, K = W.shape
        sal = group_salience(W, act_norm, g).cpu().numpy()
        bits = allocate_bits(sal, avg_bits, p)
        codes, scales, zeros = quantize_minmax(W, bits, g=g)
        return cls(pack_weights(codes, bits, g=g), bits, scales, zeros, N, K, g)

    def workspace_bytes(self, M: int) -> int:
        return workspace_bytes(M, self.N, self.K, self.bits, self.g)

    def forward(self, x: torch.Tensor, workspace: torch.Tensor, out=None) -> torch.Tensor:
        fn = mpq_gemv if x.shape[0] <= GEMV_MAX_M else mpq_gemm
        return fn(x, self.packed, self.bits, self.scales, self.zeros, self.N, workspace, out, self.g)

    def algorithmic_bytes(self, M: int) -> int:
        G = self.K // self.g
        return self.packed.numel() + 2 * 2 * G * self.N + G + 2 * M * self.K + 2 * M * self.N

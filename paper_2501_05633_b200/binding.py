"""Thin ctypes binding of include/regtopk.h: argument marshalling only.

torch is used for device memory and streams; every step of the method runs in libregtopk.so.
There is no CPU path: if the library is missing or no CUDA device is present, the calls raise.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
_ROOT = os.path.dirname(_PKG)
_SRC = os.path.join(_PKG, "csrc", "regtopk.cu")
_INC = os.path.join(_ROOT, "include")
_LIB = os.path.join(_PKG, "libregtopk.so")

OK = 0
GRAD_F32, GRAD_BF16 = 0, 1
FLAG_HOST_STAGING, FLAG_FORCE_DENSE_SELECT, FLAG_FORCE_WIDE_LISTS, FLAG_GRID_DENSE_SELECT = 1, 2, 4, 8
FLAG_NUMERATORS_AT_AGGREGATE = 16

EXPORTS = [
    "regtopk_workspace_bytes", "regtopk_create", "regtopk_worker_step", "regtopk_aggregate",
    "regtopk_global_gradient", "regtopk_state_reset", "regtopk_round_host", "regtopk_status",
    "regtopk_get_stats", "regtopk_profile_enable", "regtopk_profile_read", "regtopk_debug_residual",
    "regtopk_destroy", "regtopk_strerror", "regtopk_aggregate_pairs_static", "regtopk_aggregate_update", "regtopk_state_bytes",
    "regtopk_state_export", "regtopk_state_import", "regtopk_accumulator", "regtopk_worker_step_inplace",
    "regtopk_aggregate_gathered",
]


class Params(ctypes.Structure):
    _fields_ = [("mu", ctypes.c_float), ("omega", ctypes.POINTER(ctypes.c_float)),
                ("grad_dtype", ctypes.c_int32), ("flags", ctypes.c_int32), ("y", ctypes.c_float),
                ("n_layers", ctypes.c_int32), ("layer_end", ctypes.POINTER(ctypes.c_int64)),
                ("layer_k", ctypes.POINTER(ctypes.c_int64))]


class Stats(ctypes.Structure):
    _fields_ = [("rounds", ctypes.c_int64), ("kernel_launches", ctypes.c_int64),
                ("dense_select_workers", ctypes.c_int64), ("candidates_last", ctypes.c_int64),
                ("candidate_capacity", ctypes.c_int64), ("device_error_bits", ctypes.c_int64),
                ("post_cluster_blocks", ctypes.c_int64)]


def library_path() -> str:
    return _LIB


def build(force: bool = False, verbose: bool = False) -> str:
    """Compile csrc/regtopk.cu for sm_100a into the package directory (nvcc cross-compiles without a GPU)."""
    if not force and os.path.exists(_LIB) and os.path.getmtime(_LIB) >= max(
            os.path.getmtime(_SRC), os.path.getmtime(os.path.join(_INC, "regtopk.h"))):
        return _LIB
    cmd = ["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
           "-I", _INC, "--shared", "-Xcompiler", "-fPIC", "-o", _LIB, _SRC]
    if verbose:
        cmd.insert(1, "-Xptxas=-v")
    subprocess.run(cmd, check=True)
    return _LIB


def build_checked(force: bool = False) -> str:
    """The same library with -DREGTOPK_DEBUG=1 (every data-dependent index is range-checked on the device; a bad
    one is counted and skipped, and status() then reports an internal error), as libregtopk_checked.so beside
    the release library.  Used by tests/test_gpu_checked_build.py; nothing else loads it."""
    out = os.path.join(_PKG, "libregtopk_checked.so")
    if not force and os.path.exists(out) and os.path.getmtime(out) >= max(
            os.path.getmtime(_SRC), os.path.getmtime(os.path.join(_INC, "regtopk.h"))):
        return out
    subprocess.run(["nvcc", "-gencode", "arch=compute_100a,code=sm_100a", "-lineinfo", "-O3", "-std=c++17",
                    "-DREGTOPK_DEBUG=1", "-I", _INC, "--shared", "-Xcompiler", "-fPIC", "-o", out, _SRC], check=True)
    return out


_lib = None


def load_library():
    """dlopen the CUDA library and declare its signatures. Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB):
        raise RuntimeError(f"{_LIB} is missing: run paper_2501_05633_b200.build() (needs nvcc); "
                           "there is no CPU implementation to fall back to")
    L = ctypes.CDLL(_LIB)
    vp, i64, i32 = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int32
    L.regtopk_workspace_bytes.restype = ctypes.c_size_t
    L.regtopk_workspace_bytes.argtypes = [i64, i32, i64, ctypes.POINTER(Params)]
    L.regtopk_create.restype = ctypes.c_int
    L.regtopk_create.argtypes = [ctypes.POINTER(vp), i64, i32, i64, ctypes.POINTER(Params), vp,
                                 ctypes.c_size_t, vp]
    L.regtopk_worker_step.restype = ctypes.c_int
    L.regtopk_worker_step.argtypes = [vp, vp, i64, vp, vp]
    L.regtopk_aggregate.restype = ctypes.c_int
    L.regtopk_aggregate.argtypes = [vp, vp]
    L.regtopk_aggregate_update.restype = ctypes.c_int
    L.regtopk_aggregate_update.argtypes = [vp, vp, ctypes.c_float, vp]
    L.regtopk_aggregate_gathered.restype = ctypes.c_int
    L.regtopk_aggregate_gathered.argtypes = [vp, i32, vp, vp, ctypes.POINTER(ctypes.c_float), vp]
    L.regtopk_state_bytes.restype = ctypes.c_size_t
    L.regtopk_state_bytes.argtypes = [vp]
    L.regtopk_state_export.restype = ctypes.c_int
    L.regtopk_state_export.argtypes = [vp, vp, ctypes.c_size_t]
    L.regtopk_state_import.restype = ctypes.c_int
    L.regtopk_state_import.argtypes = [vp, vp, ctypes.c_size_t]
    L.regtopk_global_gradient.restype = ctypes.c_int
    L.regtopk_global_gradient.argtypes = [vp, ctypes.POINTER(vp)]
    L.regtopk_state_reset.restype = ctypes.c_int
    L.regtopk_state_reset.argtypes = [vp]
    L.regtopk_round_host.restype = ctypes.c_int
    L.regtopk_round_host.argtypes = [vp, vp, i64, vp, vp, vp]
    L.regtopk_status.restype = ctypes.c_int
    L.regtopk_status.argtypes = [vp]
    L.regtopk_get_stats.restype = ctypes.c_int
    L.regtopk_get_stats.argtypes = [vp, ctypes.POINTER(Stats)]
    L.regtopk_profile_enable.restype = ctypes.c_int
    L.regtopk_profile_enable.argtypes = [vp, ctypes.c_int]
    L.regtopk_profile_read.restype = ctypes.c_int
    L.regtopk_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    L.regtopk_accumulator.restype = ctypes.c_int
    L.regtopk_accumulator.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(i64)]
    L.regtopk_worker_step_inplace.restype = ctypes.c_int
    L.regtopk_worker_step_inplace.argtypes = [vp, vp, vp]
    L.regtopk_debug_residual.restype = ctypes.c_int
    L.regtopk_debug_residual.argtypes = [vp, ctypes.POINTER(vp), ctypes.POINTER(i64)]
    L.regtopk_destroy.restype = ctypes.c_int
    L.regtopk_destroy.argtypes = [vp]
    L.regtopk_aggregate_pairs_static.restype = ctypes.c_int
    L.regtopk_aggregate_pairs_static.argtypes = [i64, i32, i64, vp, vp, ctypes.POINTER(ctypes.c_float), vp, vp]
    L.regtopk_strerror.restype = ctypes.c_char_p
    L.regtopk_strerror.argtypes = [ctypes.c_int]
    _lib = L
    return L


class RegTopKError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = load_library().regtopk_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code})")


def _check(code: int, where: str):
    if code != OK:
        raise RegTopKError(code, where)


def _make_params(mu, omega, grad_dtype, flags, y=1.0, layers=None):
    """layers: None, or (layer_end, layer_k), two equally long integer sequences (see regtopk_params)."""
    p = Params()
    p.mu = float(mu)
    keep = []
    if omega is not None:
        om = (ctypes.c_float * len(omega))(*[float(x) for x in omega])
        keep.append(om)
        p.omega = ctypes.cast(om, ctypes.POINTER(ctypes.c_float))
    p.grad_dtype = grad_dtype
    p.flags = flags
    p.y = float(y)
    if layers is not None:
        ends, ks = [int(x) for x in layers[0]], [int(x) for x in layers[1]]
        if len(ends) != len(ks) or not ends:
            raise ValueError("layers = (layer_end, layer_k) of equal, non-zero length")
        e = (ctypes.c_int64 * len(ends))(*ends)
        kk = (ctypes.c_int64 * len(ks))(*ks)
        keep += [e, kk]
        p.n_layers = len(ends)
        p.layer_end = ctypes.cast(e, ctypes.POINTER(ctypes.c_int64))
        p.layer_k = ctypes.cast(kk, ctypes.POINTER(ctypes.c_int64))
    return p, keep


STATIC_SCRATCH_WORDS = 1 << 21
STATIC_MAX_WORKERS = 64


def aggregate_pairs_static(idx: torch.Tensor, val: torch.Tensor, d: int, omega=None,
                           out: Optional[torch.Tensor] = None, stream=None) -> torch.Tensor:
    """g = sum_n omega_n * ghat_n from explicit [N, k] pairs, using the library's built-in scratch
    instead of a context's workspace.  For callers that must not allocate device memory around the call:
    pass `out` (a [d] float32 device tensor made earlier) and nothing here allocates on the device.
    Calls on one GPU share the scratch; keep them on one stream or synchronise between them."""
    if not (idx.is_cuda and val.is_cuda and idx.dtype == torch.int32 and val.dtype == torch.float32):
        raise TypeError("idx int32 and val float32 device tensors [N, k]")
    idx, val = idx.contiguous(), val.contiguous()
    N, k = idx.shape
    if out is None:
        out = torch.empty(d, dtype=torch.float32, device=idx.device)
    om = None
    if omega is not None:
        om = (ctypes.c_float * N)(*[float(x) for x in omega])
    s = stream if stream is not None else torch.cuda.current_stream(idx.device)
    with torch.cuda.device(idx.device):
        _check(load_library().regtopk_aggregate_pairs_static(d, N, k, idx.data_ptr(), val.data_ptr(), om,
                                                             out.data_ptr(), s.cuda_stream),
               "regtopk_aggregate_pairs_static")
    return out


def workspace_bytes(d, N, k, mu=4.0, omega=None, grad_dtype=GRAD_F32, flags=0, y=1.0, layers=None) -> int:
    p, _keep = _make_params(mu, omega, grad_dtype, flags, y, layers)
    return int(load_library().regtopk_workspace_bytes(d, N, k, ctypes.byref(p)))


class RegTopK:
    """One (d, N, k) sparsifier context on the current CUDA device.

    grads: torch tensor [N, ld] on the device, float32 or bfloat16 as chosen at construction.
    layers = (layer_end, layer_k) selects layer by layer (regtopk_params.n_layers); k is then their sum.
    worker_step returns (idx [N,k] int32, val [N,k] float32); aggregate returns g [d] float32 (a view of
    the library's state unless `out` is given).  Work is enqueued on `stream` (default: torch's current
    stream at construction) and is asynchronous like any torch CUDA op.
    """

    def __init__(self, d: int, N: int, k: int, mu: float = 4.0, omega=None, grad_dtype=torch.float32,
                 flags: int = 0, device=None, stream: Optional[torch.cuda.Stream] = None, y: float = 1.0,
                 layers=None):
        if not torch.cuda.is_available():
            raise RuntimeError("RegTopK needs a CUDA device; there is no CPU implementation")
        self.L = load_library()
        self.device = torch.device(device if device is not None else f"cuda:{torch.cuda.current_device()}")
        self.d, self.N, self.k, self.mu = int(d), int(N), int(k), float(mu)
        self.torch_dtype = grad_dtype
        self.dtype_code = GRAD_BF16 if grad_dtype == torch.bfloat16 else GRAD_F32
        if grad_dtype not in (torch.float32, torch.bfloat16):
            raise TypeError("gradients are float32 or bfloat16")
        self.flags = int(flags)
        self.y = float(y)
        if layers is not None:  # layer-wise selection: k is the sum of the per-layer k
            k = int(sum(int(x) for x in layers[1]))
            self.k = k
        p, keep = _make_params(mu, omega, self.dtype_code, self.flags, self.y, layers)
        nbytes = int(self.L.regtopk_workspace_bytes(self.d, self.N, self.k, ctypes.byref(p)))
        if nbytes == 0:
            raise RegTopKError(-1, "regtopk_workspace_bytes")
        with torch.cuda.device(self.device):
            self.stream = stream if stream is not None else torch.cuda.current_stream()
            self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
            ctx = ctypes.c_void_p()
            _check(self.L.regtopk_create(ctypes.byref(ctx), self.d, self.N, self.k, ctypes.byref(p),
                                         self.workspace.data_ptr(), nbytes, self.stream.cuda_stream),
                   "regtopk_create")
        self.ctx = ctx
        self.workspace_nbytes = nbytes

    def close(self):
        if getattr(self, "ctx", None):
            self.L.regtopk_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check_grads(self, grads: torch.Tensor):
        if grads.dtype != self.torch_dtype or grads.dim() != 2 or grads.shape[0] != self.N:
            raise TypeError("grads must be [N, ld] of the context's dtype")
        if grads.shape[1] < self.d or grads.stride(1) != 1:
            raise ValueError("grads rows must be contiguous with ld >= d")
        return int(grads.stride(0)) if self.N > 1 else int(grads.shape[1])

    def worker_step(self, grads: torch.Tensor, out_idx: Optional[torch.Tensor] = None,
                    out_val: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        if not grads.is_cuda:
            raise TypeError("grads must live on the device (use round_host for host buffers)")
        ld = self._check_grads(grads)
        if out_idx is None:
            out_idx = torch.empty((self.N, self.k), dtype=torch.int32, device=self.device)
        if out_val is None:
            out_val = torch.empty((self.N, self.k), dtype=torch.float32, device=self.device)
        _check(self.L.regtopk_worker_step(self.ctx, grads.data_ptr(), ld, out_idx.data_ptr(),
                                          out_val.data_ptr()), "regtopk_worker_step")
        return out_idx, out_val

    def accumulator(self) -> torch.Tensor:
        """Writable view [N, d] of the library's accumulator rows: add each worker's gradient into its row
        (binary32, one addition per element), then call worker_step_inplace()."""
        ptr, ld = ctypes.c_void_p(), ctypes.c_int64()
        _check(self.L.regtopk_accumulator(self.ctx, ctypes.byref(ptr), ctypes.byref(ld)), "regtopk_accumulator")
        off = ptr.value - self.workspace.data_ptr()
        full = self.workspace[off: off + 4 * self.N * ld.value].view(torch.float32).view(self.N, ld.value)
        return full[:, : self.d]

    def worker_step_inplace(self, out_idx: Optional[torch.Tensor] = None,
                            out_val: Optional[torch.Tensor] = None) -> Tuple[torch.Tensor, torch.Tensor]:
        if out_idx is None:
            out_idx = torch.empty((self.N, self.k), dtype=torch.int32, device=self.device)
        if out_val is None:
            out_val = torch.empty((self.N, self.k), dtype=torch.float32, device=self.device)
        _check(self.L.regtopk_worker_step_inplace(self.ctx, out_idx.data_ptr(), out_val.data_ptr()),
               "regtopk_worker_step_inplace")
        return out_idx, out_val

    def aggregate(self, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        _check(self.L.regtopk_aggregate(self.ctx, out.data_ptr() if out is not None else None),
               "regtopk_aggregate")
        return out if out is not None else self.global_gradient()

    def aggregate_update(self, theta: torch.Tensor, eta: float, out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """aggregate() fused with theta <- theta - eta * g (theta: [d] float32 on the device, updated in place)."""
        if not (theta.is_cuda and theta.dtype == torch.float32 and theta.is_contiguous() and theta.numel() == self.d):
            raise TypeError("theta must be a contiguous [d] float32 device tensor")
        _check(self.L.regtopk_aggregate_update(self.ctx, theta.data_ptr(), float(eta),
                                               out.data_ptr() if out is not None else None),
               "regtopk_aggregate_update")
        return out if out is not None else self.global_gradient()

    def aggregate_gathered(self, all_idx: torch.Tensor, all_val: torch.Tensor, omega_all=None,
                           out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """aggregate() over the gathered pairs of all workers ([n_total, k] each, this context's own among them)
        when the workers are spread over several contexts (regtopk_aggregate_gathered)."""
        if not (all_idx.is_cuda and all_val.is_cuda and all_idx.dtype == torch.int32 and all_val.dtype == torch.float32
                and all_idx.is_contiguous() and all_val.is_contiguous() and all_idx.shape == all_val.shape
                and all_idx.dim() == 2 and all_idx.shape[1] == self.k):
            raise TypeError("all_idx int32 and all_val float32 contiguous device tensors [n_total, k]")
        n_total = int(all_idx.shape[0])
        om = None
        if omega_all is not None:
            if len(omega_all) != n_total:
                raise ValueError("omega_all needs one weight per gathered worker")
            om = (ctypes.c_float * n_total)(*[float(x) for x in omega_all])
        _check(self.L.regtopk_aggregate_gathered(self.ctx, n_total, all_idx.data_ptr(), all_val.data_ptr(), om,
                                                 out.data_ptr() if out is not None else None),
               "regtopk_aggregate_gathered")
        return out if out is not None else self.global_gradient()

    def state_export(self) -> torch.Tensor:
        """The state carried between rounds as one uint8 device tensor (call between rounds)."""
        n = int(self.L.regtopk_state_bytes(self.ctx))
        blob = torch.empty(n, dtype=torch.uint8, device=self.device)
        _check(self.L.regtopk_state_export(self.ctx, blob.data_ptr(), n), "regtopk_state_export")
        return blob

    def state_import(self, blob: torch.Tensor):
        if not (blob.is_cuda and blob.dtype == torch.uint8 and blob.is_contiguous()):
            raise TypeError("state blob must be a contiguous uint8 device tensor")
        _check(self.L.regtopk_state_import(self.ctx, blob.data_ptr(), blob.numel()), "regtopk_state_import")

    def global_gradient(self) -> torch.Tensor:
        """View of the library's g^t inside the workspace (overwritten by the next aggregate)."""
        ptr = ctypes.c_void_p()
        _check(self.L.regtopk_global_gradient(self.ctx, ctypes.byref(ptr)), "regtopk_global_gradient")
        off = ptr.value - self.workspace.data_ptr()
        return self.workspace[off: off + 4 * self.d].view(torch.float32)

    def residual(self) -> torch.Tensor:
        """View [N, d] of the residuals eps (test introspection)."""
        ptr, ld = ctypes.c_void_p(), ctypes.c_int64()
        _check(self.L.regtopk_debug_residual(self.ctx, ctypes.byref(ptr), ctypes.byref(ld)),
               "regtopk_debug_residual")
        off = ptr.value - self.workspace.data_ptr()
        full = self.workspace[off: off + 4 * self.N * ld.value].view(torch.float32).view(self.N, ld.value)
        return full[:, : self.d]

    def state_reset(self):
        _check(self.L.regtopk_state_reset(self.ctx), "regtopk_state_reset")

    def round_host(self, h_grads: torch.Tensor, h_idx: torch.Tensor, h_val: torch.Tensor,
                   h_g: Optional[torch.Tensor] = None):
        """A whole round from host tensors (pinned recommended); synchronises before returning."""
        if h_grads.is_cuda or h_idx.is_cuda or h_val.is_cuda:
            raise TypeError("round_host takes host tensors")
        ld = self._check_grads(h_grads)
        _check(self.L.regtopk_round_host(self.ctx, h_grads.data_ptr(), ld, h_idx.data_ptr(),
                                         h_val.data_ptr(), h_g.data_ptr() if h_g is not None else None),
               "regtopk_round_host")

    def status(self):
        _check(self.L.regtopk_status(self.ctx), "regtopk_status")

    def stats(self) -> dict:
        s = Stats()
        _check(self.L.regtopk_get_stats(self.ctx, ctypes.byref(s)), "regtopk_get_stats")
        return {n: int(getattr(s, n)) for n, _ in Stats._fields_}

    def profile_enable(self, enable: bool = True):
        _check(self.L.regtopk_profile_enable(self.ctx, 1 if enable else 0), "regtopk_profile_enable")

    def profile_read(self) -> Tuple[float, int]:
        ms, calls = ctypes.c_double(), ctypes.c_int64()
        _check(self.L.regtopk_profile_read(self.ctx, ctypes.byref(ms), ctypes.byref(calls)),
               "regtopk_profile_read")
        return float(ms.value), int(calls.value)

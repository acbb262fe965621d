"""ctypes loader and round-by-round driver for the C++ oracle.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the CPU-baseline leg of the
benchmark.  The CUDA library and its Python binding never import this module.

All arithmetic of the method lives in regtopk_oracle.cpp; this file only marshals numpy arrays and
keeps the state a training loop would keep between rounds (Algorithm 2: the residuals eps_n, the
previous mask and the accumulator values on it, and the previous aggregate g^{t-1}).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "regtopk_oracle.cpp")
_LIB = os.path.join(_HERE, "libregtopk_oracle.so")

_c_i64 = ctypes.c_int64
_c_i32 = ctypes.c_int32
_c_f32 = ctypes.c_float
_vp = ctypes.c_void_p


def build(force: bool = False) -> str:
    """Compile the oracle with g++ (no FMA contraction, no fast-math). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-std=c++17", "-O2", "-ffp-contract=off", "-fPIC", "-shared", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


def _bind(path):
    L = ctypes.CDLL(path)
    L.regtopk_oracle_tanh.restype = _c_f32
    L.regtopk_oracle_tanh.argtypes = [_c_f32]
    L.regtopk_oracle_scores.restype = None
    L.regtopk_oracle_pow.restype = _c_f32
    L.regtopk_oracle_pow.argtypes = [_c_f32, _c_f32]
    L.regtopk_oracle_scores.argtypes = [_c_i64, _vp, ctypes.c_int, _vp, _c_i64, _vp, _vp, _vp,
                                        _c_f32, _c_f32, _c_f32, _vp, _vp]
    L.regtopk_oracle_worker_step.restype = ctypes.c_int
    L.regtopk_oracle_worker_step.argtypes = [_c_i64, _c_i64, _vp, ctypes.c_int, _vp, _c_i64, _vp,
                                             _vp, _vp, _c_f32, _c_f32, _c_f32, _vp, _vp, ctypes.c_int]
    L.regtopk_oracle_worker_step_layered.restype = ctypes.c_int
    L.regtopk_oracle_worker_step_layered.argtypes = [_c_i64, _c_i64, _vp, _vp, _vp, ctypes.c_int, _vp, _c_i64, _vp,
                                                     _vp, _vp, _c_f32, _c_f32, _c_f32, _vp, _vp]
    L.regtopk_oracle_aggregate.restype = None
    L.regtopk_oracle_aggregate.argtypes = [_c_i64, _c_i32, _c_i64, _vp, _vp, _vp, _vp]
    L.regtopk_oracle_model_update.restype = None
    L.regtopk_oracle_model_update.argtypes = [_c_i64, _vp, _c_f32, _vp]
    L.regtopk_oracle_mask_certificate.restype = _c_i64
    L.regtopk_oracle_mask_certificate.argtypes = [_c_i64, _c_i64, _vp, _vp]
    return L


def _p(a):
    return None if a is None else a.ctypes.data_as(_vp)


def _grad_view(grad: np.ndarray):
    """(contiguous array, dtype code). fp32 -> 0; bf16 bit patterns carried as uint16 -> 1."""
    if grad.dtype == np.float32:
        return np.ascontiguousarray(grad), 0
    if grad.dtype == np.uint16:
        return np.ascontiguousarray(grad), 1
    raise TypeError("gradients must be float32 or uint16 (bfloat16 bit patterns)")


def _prev_views(prev_idx, prev_val, g_prev):
    if prev_idx is None or len(prev_idx) == 0:
        return 0, None, None, None
    pi = np.ascontiguousarray(prev_idx, dtype=np.int32)
    pv = np.ascontiguousarray(prev_val, dtype=np.float32)
    gp = np.ascontiguousarray(g_prev, dtype=np.float32)
    return pi.shape[0], pi, pv, gp


class OracleAPI:
    """The oracle's C functions behind numpy arguments. so_path=None builds and loads the
    in-tree source; the mutation tests pass the path of a deliberately broken build."""

    def __init__(self, so_path=None):
        self.L = _bind(so_path or build())

    def tanh_spec(self, x) -> np.ndarray:
        x = np.asarray(x, dtype=np.float32)
        out = np.empty_like(x)
        fi, fo = x.reshape(-1), out.reshape(-1)
        for i in range(fi.size):
            fo[i] = self.L.regtopk_oracle_tanh(_c_f32(float(fi[i])))
        return out

    def pow_spec(self, m, p) -> np.ndarray:
        m = np.asarray(m, dtype=np.float32)
        out = np.empty_like(m)
        fi, fo = m.reshape(-1), out.reshape(-1)
        for i in range(fi.size):
            fo[i] = self.L.regtopk_oracle_pow(_c_f32(float(fi[i])), _c_f32(float(p)))
        return out

    def scores(self, grad, eps, prev_idx, prev_val, g_prev, mu, omega_n, y=1.0):
        """(a, score) of one worker; prev_idx=None means no previous round."""
        grad, code = _grad_view(grad)
        d = grad.shape[0]
        eps = np.ascontiguousarray(eps, dtype=np.float32)
        a = np.empty(d, np.float32)
        s = np.empty(d, np.float32)
        n_prev, pi, pv, gp = _prev_views(prev_idx, prev_val, g_prev)
        self.L.regtopk_oracle_scores(d, _p(grad), code, _p(eps), n_prev, _p(pi), _p(pv), _p(gp),
                                     mu, omega_n, y, _p(a), _p(s))
        return a, s

    def worker_step(self, grad, eps, k, prev_idx, prev_val, g_prev, mu, omega_n, select_mode=0, y=1.0):
        """One worker, one round. eps (float32, contiguous) is updated in place. Returns (idx, val)."""
        grad, code = _grad_view(grad)
        d = grad.shape[0]
        assert eps.dtype == np.float32 and eps.flags.c_contiguous and eps.shape == (d,)
        out_idx = np.empty(k, np.int32)
        out_val = np.empty(k, np.float32)
        n_prev, pi, pv, gp = _prev_views(prev_idx, prev_val, g_prev)
        rc = self.L.regtopk_oracle_worker_step(d, k, _p(grad), code, _p(eps), n_prev, _p(pi),
                                               _p(pv), _p(gp), mu, omega_n, y, _p(out_idx),
                                               _p(out_val), select_mode)
        if rc != 0:
            raise ValueError("oracle rejected the arguments (need 1 <= k <= d < 2^31, 0 < y <= 1)")
        return out_idx, out_val

    def worker_step_layered(self, grad, eps, seg_end, seg_k, prev_idx, prev_val, g_prev, mu, omega_n, y=1.0):
        """One worker, one round, with one Top-k per layer: layer l is [seg_end[l-1], seg_end[l]) and keeps seg_k[l]
        entries.  eps is updated in place.  Returns (idx, val) with sum(seg_k) pairs in ascending index order."""
        grad, code = _grad_view(grad)
        d = grad.shape[0]
        assert eps.dtype == np.float32 and eps.flags.c_contiguous and eps.shape == (d,)
        se = np.ascontiguousarray(seg_end, dtype=np.int64)
        sk = np.ascontiguousarray(seg_k, dtype=np.int64)
        K = int(sk.sum())
        out_idx = np.empty(K, np.int32)
        out_val = np.empty(K, np.float32)
        n_prev, pi, pv, gp = _prev_views(prev_idx, prev_val, g_prev)
        rc = self.L.regtopk_oracle_worker_step_layered(d, se.shape[0], _p(se), _p(sk), _p(grad), code, _p(eps), n_prev,
                                                       _p(pi), _p(pv), _p(gp), mu, omega_n, y, _p(out_idx), _p(out_val))
        if rc != 0:
            raise ValueError("oracle rejected the layer table (ascending ends, last == d, 1 <= k_l <= layer size)")
        return out_idx, out_val

    def aggregate(self, d, omega, idx, val):
        idx = np.ascontiguousarray(idx, dtype=np.int32)
        val = np.ascontiguousarray(val, dtype=np.float32)
        omega = np.ascontiguousarray(omega, dtype=np.float32)
        N, k = idx.shape
        g = np.empty(d, np.float32)
        self.L.regtopk_oracle_aggregate(d, N, k, _p(omega), _p(idx), _p(val), _p(g))
        return g

    def model_update(self, theta, eta, g):
        """theta <- theta - eta * g in place (theta float32, contiguous)."""
        assert theta.dtype == np.float32 and theta.flags.c_contiguous
        g = np.ascontiguousarray(g, dtype=np.float32)
        self.L.regtopk_oracle_model_update(theta.shape[0], _p(theta), eta, _p(g))
        return theta

    def mask_certificate(self, score, sel_idx):
        score = np.ascontiguousarray(score, dtype=np.float32)
        sel_idx = np.ascontiguousarray(sel_idx, dtype=np.int32)
        return int(self.L.regtopk_oracle_mask_certificate(score.shape[0], sel_idx.shape[0],
                                                          _p(score), _p(sel_idx)))


_default = None


def default() -> OracleAPI:
    global _default
    if _default is None:
        _default = OracleAPI()
    return _default


def grads_view(grads_cpu, d: int) -> np.ndarray:
    """[N, ld] torch CPU tensor -> [N, d] numpy array the oracle reads (bfloat16 as uint16 bit patterns)."""
    import torch
    if grads_cpu.dtype == torch.bfloat16:
        return np.ascontiguousarray(grads_cpu.view(torch.int16).numpy().view(np.uint16)[:, :d])
    return np.ascontiguousarray(grads_cpu.numpy()[:, :d])


class OracleRegTopK:
    """State of N workers and the server across rounds (Algorithm 2's initialisation and loop).

    worker_step(grads) runs every worker's round; aggregate() runs the server and rolls the state
    (previous mask/values <- this round's pairs, g_prev <- g, round += 1).  threads > 1 only spreads
    independent workers over host threads; each worker's computation is unchanged.
    """

    def __init__(self, d, N, k, mu, omega=None, select_mode=0, threads=1, api=None, y=1.0, layers=None):
        """layers: None, or (seg_end, seg_k) for one Top-k per layer; k is then ignored and becomes sum(seg_k)."""
        self.api = api or default()
        self.y = float(y)
        self.layers = None
        if layers is not None:
            self.layers = (np.asarray(layers[0], np.int64).copy(), np.asarray(layers[1], np.int64).copy())
            k = int(self.layers[1].sum())
        self.d, self.N, self.k, self.mu = int(d), int(N), int(k), float(mu)
        self.omega = (np.full(N, np.float32(1.0) / np.float32(N), np.float32) if omega is None
                      else np.asarray(omega, np.float32).copy())
        self.select_mode = select_mode
        self.threads = threads
        self.reset()

    def reset(self):
        self.eps = np.zeros((self.N, self.d), np.float32)  # eps_n^0 = 0
        self.round = 0
        self.prev_idx = None
        self.prev_val = None
        self.g_prev = None
        self.idx = None
        self.val = None

    def _one(self, n, grads):
        pi = None if self.prev_idx is None else self.prev_idx[n]
        pv = None if self.prev_val is None else self.prev_val[n]
        if self.layers is not None:
            return self.api.worker_step_layered(grads[n], self.eps[n], self.layers[0], self.layers[1], pi, pv,
                                                self.g_prev, self.mu, float(self.omega[n]), self.y)
        return self.api.worker_step(grads[n], self.eps[n], self.k, pi, pv, self.g_prev, self.mu,
                           float(self.omega[n]), self.select_mode, self.y)

    def worker_step(self, grads):
        assert grads.shape == (self.N, self.d)
        if self.threads > 1:
            with ThreadPoolExecutor(self.threads) as ex:
                res = list(ex.map(lambda n: self._one(n, grads), range(self.N)))
        else:
            res = [self._one(n, grads) for n in range(self.N)]
        self.idx = np.stack([r[0] for r in res])
        self.val = np.stack([r[1] for r in res])
        return self.idx, self.val

    def aggregate(self):
        g = self.api.aggregate(self.d, self.omega, self.idx, self.val)
        self.prev_idx, self.prev_val, self.g_prev = self.idx, self.val, g
        self.round += 1
        return g

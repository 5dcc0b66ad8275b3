"""ctypes binding of libvcas.so: one Python function per C entry point of include/vcas.h.

Argument marshalling only: torch tensors provide device memory and the current CUDA stream,
every step of the method runs in the library's kernels.  If the compiled library is missing
this module raises on first use; there is no other implementation to fall back to.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libvcas.so")

VCAS_OK = 0
ERRORS = {-1: "VCAS_ERR_BAD_ARG", -2: "VCAS_ERR_SHAPE", -3: "VCAS_ERR_DTYPE", -4: "VCAS_ERR_WORKSPACE",
          -5: "VCAS_ERR_CUDA", -6: "VCAS_ERR_TIMEOUT", -7: "VCAS_ERR_INTERNAL"}
DTYPE_F32, DTYPE_BF16 = 0, 1
GEMM_AUTO, GEMM_FMA, GEMM_TENSOR = 0, 1, 2

EXPORTS = ["vcas_default_config", "vcas_create", "vcas_destroy", "vcas_workspace_bytes", "vcas_linear_bwd",
           "vcas_linear_bwd_ex", "vcas_linear_bwd_chain", "vcas_chain_parts", "vcas_layernorm_bwd", "vcas_join", "vcas_dense_bwd", "vcas_dense_bwd_ex", "vcas_score", "vcas_last_sampling", "vcas_mask_from_probs",
           "vcas_variance_probe", "vcas_update_ratios", "vcas_last_device_status", "vcas_launch_count",
           "vcas_set_profiling", "vcas_stage_times", "vcas_set_wait_limit",
           "vcas_set_probe_subsample", "vcas_get_probe_subsample", "vcas_score_static", "vcas_set_tuning",
           "vcas_last_plan", "vcas_version"]


class VcasError(RuntimeError):
    def __init__(self, code: int, where: str):
        super().__init__(f"{where} failed: {ERRORS.get(code, code)}")
        self.code = code


class LayerDesc(C.Structure):
    _fields_ = [("N", C.c_int32), ("T", C.c_int32), ("d_in", C.c_int32), ("d_out", C.c_int32),
                ("dtype", C.c_int32), ("gemm_path", C.c_int32)]


class Config(C.Structure):
    _fields_ = [("F", C.c_int32), ("M", C.c_int32), ("tau_act", C.c_float), ("tau_w", C.c_float),
                ("alpha", C.c_float), ("beta", C.c_float), ("rho_min", C.c_float), ("nu_min", C.c_float)]


class State(C.Structure):
    _fields_ = [("s", C.c_float), ("t", C.c_int32), ("L", C.c_int32),
                ("rho", C.POINTER(C.c_float)), ("nu", C.POINTER(C.c_float))]


class ChainArgs(C.Structure):
    _fields_ = [("H", C.c_void_p), ("a_in", C.c_void_p), ("a_in_parts", C.c_int32), ("alive_in", C.c_void_p),
                ("alive_cnt_in", C.c_void_p), ("a_out", C.c_void_p), ("kept_out", C.c_void_p),
                ("kept_cnt_out", C.c_void_p), ("skip_dropped_rows", C.c_int32), ("defer_join", C.c_int32)]


_lib = None


def lib() -> C.CDLL:
    """Loads libvcas.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2402_17227_b200.build` (needs nvcc); "
                               "there is no CPU implementation")
        l = C.CDLL(LIB_PATH)
        for name in EXPORTS:
            getattr(l, name).restype = C.c_int
        _lib = l
    return _lib


def _check(code: int, where: str) -> None:
    if code != VCAS_OK:
        raise VcasError(code, where)


def _ptr(t):
    if t is None:
        return C.c_void_p(None)
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def default_config() -> Config:
    cfg = Config()
    _check(lib().vcas_default_config(C.byref(cfg)), "vcas_default_config")
    return cfg


@dataclass
class Sampling:
    g: torch.Tensor
    p: torch.Tensor
    w: torch.Tensor
    q: torch.Tensor
    idxA: torch.Tensor
    cntA: int
    idxW: torch.Tensor
    cntW: int


class Layer:
    """A handle for one layer shape (vcas_create / vcas_destroy) on the current CUDA device."""

    def __init__(self, N: int, T: int, d_in: int, d_out: int, dtype: torch.dtype = torch.bfloat16,
                 gemm_path: int = GEMM_AUTO, config: Config | None = None):
        if not torch.cuda.is_available():
            raise RuntimeError("libvcas needs a CUDA device (sm_100a); there is no CPU path")
        self.N, self.T, self.d_in, self.d_out, self.dtype = N, T, d_in, d_out, dtype
        self.R = N * T
        self.config = config if config is not None else default_config()
        desc = LayerDesc(N, T, d_in, d_out, {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[dtype], gemm_path)
        self._h = C.c_void_p(None)
        _check(lib().vcas_create(C.byref(self._h), C.byref(desc), C.byref(self.config)), "vcas_create")

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h.value:
            lib().vcas_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ products
    def _outs(self, dX, dW, dev):
        if dX is None:
            dX = torch.empty(self.R, self.d_in, dtype=self.dtype, device=dev)
        if dW is None:
            dW = torch.empty(self.d_out, self.d_in, dtype=torch.float32, device=dev)
        return dX, dW

    def linear_bwd(self, X, dY, W, rho: float, nu: float, seed: int, *, p_in=None, q_in=None, H=None,
                   dX=None, dW=None):
        dX, dW = self._outs(dX, dW, X.device)
        rc = lib().vcas_linear_bwd_ex(self._h, _ptr(X), _ptr(dY), _ptr(W), C.c_float(rho), C.c_float(nu),
                                      C.c_uint64(seed), _ptr(p_in), _ptr(q_in), _ptr(H), _ptr(dX), _ptr(dW),
                                      _stream())
        _check(rc, "vcas_linear_bwd_ex")
        return dX, dW

    def linear_bwd_chain(self, X, dY, W, rho: float, nu: float, seed: int, dX, dW, *, H=None, a_in=None,
                         a_in_parts: int = 1, alive_in=None, alive_cnt_in=None, a_out=None, kept_out=None,
                         kept_cnt_out=None, skip_dropped_rows: bool = False, defer_join: bool = False):
        """vcas_linear_bwd_chain: scores handed down from the layer above (a_in, alive_in) and to the layer
        below (a_out, kept_out); every extra is an optional device tensor."""
        dp = lambda t: None if t is None else t.data_ptr()
        args = ChainArgs(dp(H), dp(a_in), a_in_parts, dp(alive_in), dp(alive_cnt_in), dp(a_out), dp(kept_out),
                         dp(kept_cnt_out), 1 if skip_dropped_rows else 0, 1 if defer_join else 0)
        _check(lib().vcas_linear_bwd_chain(self._h, _ptr(X), _ptr(dY), _ptr(W), C.c_float(rho), C.c_float(nu),
                                           C.c_uint64(seed), C.byref(args), _ptr(dX), _ptr(dW), _stream()),
               "vcas_linear_bwd_chain")

    def layernorm_bwd(self, X, gamma, dY, rho: float, seed: int, eps: float = 1e-5, *, dX=None, a_in=None,
                      a_in_parts: int = 1, alive_in=None, alive_cnt_in=None, a_out=None, kept_out=None,
                      kept_cnt_out=None, skip_dropped_rows: bool = False):
        """vcas_layernorm_bwd on a handle made with d_in = d_out = the normalised width.  Returns (dX, dgamma, dbeta)."""
        dev = X.device
        if dX is None:
            dX = torch.empty(self.R, self.d_in, dtype=self.dtype, device=dev)
        dg = torch.empty(self.d_in, dtype=torch.float32, device=dev)
        db = torch.empty(self.d_in, dtype=torch.float32, device=dev)
        dp = lambda t: None if t is None else t.data_ptr()
        args = ChainArgs(None, dp(a_in), a_in_parts, dp(alive_in), dp(alive_cnt_in), dp(a_out), dp(kept_out),
                         dp(kept_cnt_out), 1 if skip_dropped_rows else 0, 0)
        _check(lib().vcas_layernorm_bwd(self._h, _ptr(X), _ptr(gamma), _ptr(dY), C.c_float(eps), C.c_float(rho),
                                        C.c_uint64(seed), C.byref(args), _ptr(dX), _ptr(dg), _ptr(db), _stream()),
               "vcas_layernorm_bwd")
        return dX, dg, db

    def join(self) -> None:
        _check(lib().vcas_join(self._h, _stream()), "vcas_join")

    def chain_parts(self) -> int:
        n = C.c_int32(0)
        _check(lib().vcas_chain_parts(self._h, C.byref(n)), "vcas_chain_parts")
        return n.value

    def linear_bwd_plain(self, X, dY, W, rho: float, nu: float, seed: int, dX, dW):
        """vcas_linear_bwd with caller-provided outputs (the call a training loop makes)."""
        _check(lib().vcas_linear_bwd(self._h, _ptr(X), _ptr(dY), _ptr(W), C.c_float(rho), C.c_float(nu),
                                     C.c_uint64(seed), _ptr(dX), _ptr(dW), _stream()), "vcas_linear_bwd")

    def dense_bwd(self, X, dY, W, *, H=None, dX=None, dW=None):
        dX, dW = self._outs(dX, dW, X.device)
        _check(lib().vcas_dense_bwd_ex(self._h, _ptr(X), _ptr(dY), _ptr(W), _ptr(H), _ptr(dX), _ptr(dW), _stream()),
               "vcas_dense_bwd_ex")
        return dX, dW

    # ------------------------------------------------------------------ sampling
    def _sampling_buffers(self, dev):
        f = dict(dtype=torch.float32, device=dev)
        i = dict(dtype=torch.int32, device=dev)
        return (torch.empty(self.N, **f), torch.empty(self.N, **f), torch.empty(self.R, **f),
                torch.empty(self.R, **f), torch.empty(self.N, **i), torch.zeros(1, **i),
                torch.empty(self.R, **i), torch.zeros(1, **i))

    @staticmethod
    def _pack_sampling(b) -> Sampling:
        g, p, w, q, idxA, cntA, idxW, cntW = b
        ca, cw = int(cntA.item()), int(cntW.item())
        return Sampling(g, p, w, q, idxA[:ca], ca, idxW[:cw], cw)

    def score(self, X, dY, rho: float, nu: float, seed: int) -> Sampling:
        b = self._sampling_buffers(X.device)
        _check(lib().vcas_score(self._h, _ptr(X), _ptr(dY), C.c_float(rho), C.c_float(nu), C.c_uint64(seed),
                                *[_ptr(t) for t in b], _stream()), "vcas_score")
        return self._pack_sampling(b)

    def last_sampling(self, device=None) -> Sampling:
        b = self._sampling_buffers(device or torch.device("cuda", torch.cuda.current_device()))
        _check(lib().vcas_last_sampling(self._h, *[_ptr(t) for t in b], _stream()), "vcas_last_sampling")
        return self._pack_sampling(b)

    def mask_from_probs(self, p, seed: int, sampler_id: int):
        n = p.numel()
        keep = torch.empty(n, dtype=torch.uint8, device=p.device)
        idx = torch.empty(n, dtype=torch.int32, device=p.device)
        cnt = torch.zeros(1, dtype=torch.int32, device=p.device)
        _check(lib().vcas_mask_from_probs(self._h, _ptr(p), C.c_int32(n), C.c_uint64(seed), C.c_int32(sampler_id),
                                          _ptr(keep), _ptr(idx), _ptr(cnt), _stream()), "vcas_mask_from_probs")
        c = int(cnt.item())
        return keep, idx[:c], c

    # --------------------------------------------------------------------- probe
    def variance_probe(self, Xs, dYs, W, rho: float, nu: float, s: float, seed: int, out=None):
        """Returns a device tensor [V_s, V_act, V_w, p_lo, p_hi] (fp32), filled asynchronously."""
        M = len(Xs)
        if out is None:
            out = torch.zeros(5, dtype=torch.float32, device=W.device)
        xa = (C.c_void_p * M)(*[x.data_ptr() for x in Xs])
        ya = (C.c_void_p * M)(*[y.data_ptr() for y in dYs])
        base, st = out.data_ptr(), 4
        rc = lib().vcas_variance_probe(self._h, C.c_int32(M), xa, ya, _ptr(W), C.c_float(rho), C.c_float(nu),
                                       C.c_float(s), C.c_uint64(seed), *[C.c_void_p(base + st * k) for k in range(5)],
                                       _stream())
        _check(rc, "vcas_variance_probe")
        return out

    # ---------------------------------------------------------------------- misc
    def device_status(self) -> int:
        st = C.c_int32(0)
        _check(lib().vcas_last_device_status(self._h, C.byref(st)), "vcas_last_device_status")
        return st.value

    def set_tuning(self, dx_tile_n: int = 0, dw_tile_n: int = 0, dx_split_k: int = 0, dw_split_k: int = 0,
                   tile_m: int = 0, dw_tile_m: int | None = None) -> None:
        """tile_m: tile height of the dX product, and of the dW product too unless dw_tile_m is given."""
        _check(lib().vcas_set_tuning(self._h, C.c_int32(dx_tile_n), C.c_int32(dw_tile_n), C.c_int32(dx_split_k),
                                     C.c_int32(dw_split_k), C.c_int32(tile_m),
                                     C.c_int32(tile_m if dw_tile_m is None else dw_tile_m)), "vcas_set_tuning")

    def last_plan(self):
        """((width, slices, height code) of the dX product, the same of the dW product) of the last call."""
        a = (C.c_int32 * 6)()
        _check(lib().vcas_last_plan(self._h, a), "vcas_last_plan")
        return tuple(a[0:3]), tuple(a[3:6])

    def set_probe_subsample(self, rows: int, seed: int = 0) -> None:
        _check(lib().vcas_set_probe_subsample(self._h, C.c_int32(rows), C.c_uint64(seed)), "vcas_set_probe_subsample")

    def probe_subsample(self):
        """The rows of the parameter gradient the probe samples (host list; empty when it uses all rows)."""
        n = C.c_int32(0)
        _check(lib().vcas_get_probe_subsample(self._h, None, C.byref(n)), "vcas_get_probe_subsample")
        rows = (C.c_int32 * max(1, n.value))()
        _check(lib().vcas_get_probe_subsample(self._h, rows, C.byref(n)), "vcas_get_probe_subsample")
        return list(rows)[:n.value]

    def set_wait_limit(self, limit_ns: int, stall_once: bool = False) -> None:
        _check(lib().vcas_set_wait_limit(self._h, C.c_uint64(limit_ns), C.c_int32(1 if stall_once else 0)),
               "vcas_set_wait_limit")

    def set_profiling(self, enable: bool) -> None:
        _check(lib().vcas_set_profiling(self._h, C.c_int32(1 if enable else 0)), "vcas_set_profiling")

    def stage_times(self):
        """(ms[8], calls[2]) summed over the calls recorded since profiling was enabled or last read."""
        ms = (C.c_float * 8)()
        calls = (C.c_int32 * 2)()
        _check(lib().vcas_stage_times(self._h, ms, calls), "vcas_stage_times")
        return list(ms), list(calls)

    def launch_count(self) -> int:
        n = C.c_uint64(0)
        _check(lib().vcas_launch_count(self._h, C.byref(n)), "vcas_launch_count")
        return n.value

    def workspace_bytes(self) -> int:
        n = C.c_size_t(0)
        _check(lib().vcas_workspace_bytes(self._h, C.byref(n)), "vcas_workspace_bytes")
        return n.value


def update_ratios(s: float, rho, nu, V_s, V_act, V_w, p_lo, p_hi, config: Config, t: int = 0):
    """vcas_update_ratios on host lists of length L; returns (s, rho, nu)."""
    L = len(rho)
    arr = lambda v: (C.c_float * L)(*[float(x) for x in v])
    rho_a, nu_a = arr(rho), arr(nu)
    st = State(float(s), int(t), L, C.cast(rho_a, C.POINTER(C.c_float)), C.cast(nu_a, C.POINTER(C.c_float)))
    rc = lib().vcas_update_ratios(C.byref(st), C.c_int32(L), arr(V_s), arr(V_act), arr(V_w), arr(p_lo), arr(p_hi),
                                  C.byref(config))
    _check(rc, "vcas_update_ratios")
    return st.s, list(rho_a), list(nu_a)


def score_static(X, dY, N: int, T: int, rho: float, nu: float, seed: int) -> Sampling:
    """vcas_score_static: scores, probabilities and index lists without a handle or any device
    allocation by the library (the output tensors below are the caller's, made by torch).
    Limits: N <= 4096, N*T <= 16384.  Calls sharing a device must not overlap on the GPU."""
    R, dev = N * T, X.device
    f = dict(dtype=torch.float32, device=dev)
    i = dict(dtype=torch.int32, device=dev)
    b = (torch.empty(N, **f), torch.empty(N, **f), torch.empty(R, **f), torch.empty(R, **f),
         torch.empty(N, **i), torch.zeros(1, **i), torch.empty(R, **i), torch.zeros(1, **i))
    dt = {torch.float32: DTYPE_F32, torch.bfloat16: DTYPE_BF16}[X.dtype]
    rc = lib().vcas_score_static(C.c_int32(N), C.c_int32(T), C.c_int32(X.shape[1]), C.c_int32(dY.shape[1]),
                                 C.c_int32(dt), _ptr(X), _ptr(dY), C.c_float(rho), C.c_float(nu), C.c_uint64(seed),
                                 *[_ptr(t) for t in b], _stream())
    _check(rc, "vcas_score_static")
    return Layer._pack_sampling(b)


def version() -> int:
    return lib().vcas_version()

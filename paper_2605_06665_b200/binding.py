"""ctypes binding of libunipool.so - argument marshalling only.

Every function here forwards to the C-ABI entry point of the same name declared
in include/unipool.h; PyTorch supplies device memory (``tensor.data_ptr()``) and
the current CUDA stream.  There is no CPU fallback: if the library is missing
or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libunipool.so")

FP32, BF16 = 0, 1
ROUTER_NORM, ROUTER_SOFTMAX = 0, 1
ROW_ALIGN = 128
BWD_SKIP_WGRAD = 1
WGRAD_OVERWRITE = 2

EXPORTS = (
    "unipool_row_capacity", "unipool_workspace_bytes", "unipool_create", "unipool_destroy",
    "unipool_last_error", "unipool_check_status", "unipool_route", "unipool_dispatch",
    "unipool_expert_fwd", "unipool_combine", "unipool_expert_bwd", "unipool_pool_wgrad",
    "unipool_pool_aux_loss", "unipool_route_bwd", "unipool_calibrate_c",
    "unipool_profile_enable", "unipool_profile_read", "unipool_dispatch_static",
    "unipool_unique_experts", "unipool_router_prepare", "unipool_selftest_wait",
)

PHASES = (
    "route_logits", "route_select", "dispatch_maps", "dispatch_gather", "expert_fwd_gu", "expert_fwd_down",
    "combine", "pool_aux", "bwd_scale_gather", "bwd_dgate", "dgrad_down", "dgrad_gu", "wgrad_down", "wgrad_gu",
    "unpermute_sum", "route_bwd_dz", "route_bwd_dx", "route_bwd_dw",
)


class Config(ctypes.Structure):
    _fields_ = [
        ("d_model", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("pool_size", ctypes.c_int32),
        ("top_k", ctypes.c_int32), ("n_layers", ctypes.c_int32), ("max_tokens", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("eps", ctypes.c_float), ("c", ctypes.c_float),
        ("router_mode", ctypes.c_int32),
    ]


class UniPoolError(RuntimeError):
    def __init__(self, code, message):
        super().__init__(f"unipool error {code}: {message}")
        self.code = code


_lib = None


def lib():
    """Loads libunipool.so once; raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(
            f"{LIB_PATH} is missing: build it with `python -m paper_2605_06665_b200.build` "
            "(there is no CPU fallback)")
    L = ctypes.CDLL(LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    cfgp = ctypes.POINTER(Config)
    L.unipool_row_capacity.restype = i64
    L.unipool_row_capacity.argtypes = [cfgp]
    L.unipool_workspace_bytes.restype = ctypes.c_size_t
    L.unipool_workspace_bytes.argtypes = [cfgp]
    L.unipool_create.restype = ctypes.c_int
    L.unipool_create.argtypes = [ctypes.POINTER(vp), cfgp, vp, ctypes.c_size_t, vp]
    L.unipool_destroy.restype = ctypes.c_int
    L.unipool_destroy.argtypes = [vp]
    L.unipool_last_error.restype = ctypes.c_char_p
    L.unipool_last_error.argtypes = []
    L.unipool_check_status.restype = ctypes.c_int
    L.unipool_check_status.argtypes = [vp, vp]
    L.unipool_route.restype = ctypes.c_int
    L.unipool_route.argtypes = [vp, vp, i32, vp, f32, vp, i32, vp, vp, vp, vp, vp, vp, vp]
    L.unipool_router_prepare.restype = ctypes.c_int
    L.unipool_router_prepare.argtypes = [vp, vp, i32, i32, vp]
    L.unipool_dispatch.restype = ctypes.c_int
    L.unipool_dispatch.argtypes = [vp, vp, i32, vp, i32, vp, vp, vp, vp, vp, vp]
    L.unipool_dispatch_static.restype = ctypes.c_int
    L.unipool_dispatch_static.argtypes = [vp, i32, i32, i32, i32, vp, i32, i64, vp, vp, vp, vp, vp, vp]
    L.unipool_expert_fwd.restype = ctypes.c_int
    L.unipool_expert_fwd.argtypes = [vp, vp, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp]
    L.unipool_combine.restype = ctypes.c_int
    L.unipool_combine.argtypes = [vp, vp, vp, vp, i32, vp, vp, vp]
    L.unipool_expert_bwd.restype = ctypes.c_int
    L.unipool_expert_bwd.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, i32, i32,
                                     vp, vp, vp, vp, vp, vp, vp, i32, vp]
    L.unipool_pool_wgrad.restype = ctypes.c_int
    L.unipool_pool_wgrad.argtypes = [vp, i32, i64, vp, vp, vp, vp, vp, i32, i32, vp, vp, i32, vp]
    L.unipool_pool_aux_loss.restype = ctypes.c_int
    L.unipool_pool_aux_loss.argtypes = [vp, vp, vp, i32, i32, i32, f32, vp, vp, vp, vp, vp]
    L.unipool_route_bwd.restype = ctypes.c_int
    L.unipool_route_bwd.argtypes = [vp, vp, i32, vp, f32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    L.unipool_unique_experts.restype = ctypes.c_int
    L.unipool_unique_experts.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp]
    L.unipool_calibrate_c.restype = ctypes.c_int
    L.unipool_calibrate_c.argtypes = [vp, i32, i32, i32, ctypes.c_uint64, ctypes.POINTER(f32), vp]
    L.unipool_selftest_wait.restype = ctypes.c_int
    L.unipool_selftest_wait.argtypes = [vp, i64, vp]
    L.unipool_profile_enable.restype = ctypes.c_int
    L.unipool_profile_enable.argtypes = [vp, i32]
    L.unipool_profile_read.restype = ctypes.c_int
    L.unipool_profile_read.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
    _lib = L
    return L


def _check(rc):
    if rc != 0:
        raise UniPoolError(rc, lib().unipool_last_error().decode())


def _p(t):
    """Device pointer of a tensor (None -> NULL)."""
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream():
    import torch
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_config(d_model, d_ff, pool_size, top_k, n_layers, max_tokens, dtype, eps, c, router_mode=0):
    return Config(d_model, d_ff, pool_size, top_k, n_layers, max_tokens, dtype, eps, c, router_mode)


def row_capacity(cfg):
    return int(lib().unipool_row_capacity(ctypes.byref(cfg)))


def workspace_bytes(cfg):
    return int(lib().unipool_workspace_bytes(ctypes.byref(cfg)))


def dispatch_static(x, T, d_model, dtype, top_k, idx, n_experts, row_capacity, offsets, row_of, token_of,
                    tile_expert, Xp):
    """unipool_dispatch_static: the token permute for callers without a workspace or a context
    (its scratch is built into the library; it allocates nothing)."""
    _check(lib().unipool_dispatch_static(_p(x), T, d_model, dtype, top_k, _p(idx), n_experts, row_capacity,
                                         _p(offsets), _p(row_of), _p(token_of), _p(tile_expert), _p(Xp),
                                         _stream()))


class Context:
    """Owns a unipool_ctx and the torch tensor that backs its workspace."""

    def __init__(self, cfg, device="cuda"):
        import torch
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = workspace_bytes(cfg)
        if nbytes == 0:
            # let unipool_create produce the precise message
            nbytes = 256
        self.workspace = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        self.handle = ctypes.c_void_p()
        _check(lib().unipool_create(ctypes.byref(self.handle), ctypes.byref(cfg), _p(self.workspace),
                                    self.workspace.numel(), _stream()))
        self.row_capacity = row_capacity(cfg)

    def close(self):
        if self.handle:
            lib().unipool_destroy(self.handle)
            self.handle = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- one method per C entry point, same names, same argument order ----
    def check_status(self):
        _check(lib().unipool_check_status(self.handle, _stream()))

    def route(self, x, T, W_r, sigma, bias, n_experts, idx, gate, counts, score_sum, znorm, z_saved):
        _check(lib().unipool_route(self.handle, _p(x), T, _p(W_r), sigma, _p(bias), n_experts, _p(idx),
                                   _p(gate), _p(counts), _p(score_sum), _p(znorm), _p(z_saved), _stream()))

    def selftest_wait(self, limit_cycles):
        _check(lib().unipool_selftest_wait(self.handle, int(limit_cycles), _stream()))

    def router_prepare(self, W_r, n_layers, n_experts):
        _check(lib().unipool_router_prepare(self.handle, _p(W_r), n_layers, n_experts, _stream()))

    def dispatch(self, x, T, idx, n_experts, offsets, row_of, token_of, tile_expert, Xp):
        _check(lib().unipool_dispatch(self.handle, _p(x), T, _p(idx), n_experts, _p(offsets), _p(row_of),
                                      _p(token_of), _p(tile_expert), _p(Xp), _stream()))

    def expert_fwd(self, Xp, offsets, tile_expert, W_gu, W_down, expert_base, n_experts, GU, A, Yp):
        _check(lib().unipool_expert_fwd(self.handle, _p(Xp), _p(offsets), _p(tile_expert), _p(W_gu),
                                        _p(W_down), expert_base, n_experts, _p(GU), _p(A), _p(Yp), _stream()))

    def combine(self, Yp, row_of, gate, T, residual, y):
        _check(lib().unipool_combine(self.handle, _p(Yp), _p(row_of), _p(gate), T, _p(residual), _p(y),
                                     _stream()))

    def expert_bwd(self, dy, T, row_of, gate, token_of, offsets, tile_expert, Xp, GU, A, Yp, W_gu, W_down,
                   expert_base, n_experts, dx_residual, dYp, dGU, dx, dgate, dW_gu, dW_down, flags=0):
        _check(lib().unipool_expert_bwd(self.handle, _p(dy), T, _p(row_of), _p(gate), _p(token_of),
                                        _p(offsets), _p(tile_expert), _p(Xp), _p(GU), _p(A), _p(Yp),
                                        _p(W_gu), _p(W_down), expert_base, n_experts, _p(dx_residual),
                                        _p(dYp), _p(dGU), _p(dx), _p(dgate), _p(dW_gu), _p(dW_down),
                                        flags, _stream()))

    def pool_wgrad(self, n_layers, layer_stride_rows, offsets, Xp, A, dYp, dGU, expert_base, n_experts,
                   dW_gu, dW_down, flags=0):
        _check(lib().unipool_pool_wgrad(self.handle, n_layers, layer_stride_rows, _p(offsets), _p(Xp), _p(A),
                                        _p(dYp), _p(dGU), expert_base, n_experts, _p(dW_gu), _p(dW_down),
                                        flags, _stream()))

    def pool_aux_loss(self, counts, score_sum, L, n_experts, T, alpha, fbar_prev, loss, dscore_coef, fbar_out):
        _check(lib().unipool_pool_aux_loss(self.handle, _p(counts), _p(score_sum), L, n_experts, T, alpha,
                                           _p(fbar_prev), _p(loss), _p(dscore_coef), _p(fbar_out), _stream()))

    def route_bwd(self, x, T, W_r, sigma, n_experts, znorm, z_saved, idx, dgate, dscore_coef, dx, dW_r, dsigma):
        _check(lib().unipool_route_bwd(self.handle, _p(x), T, _p(W_r), sigma, n_experts, _p(znorm),
                                       _p(z_saved), _p(idx), _p(dgate), _p(dscore_coef), _p(dx), _p(dW_r),
                                       _p(dsigma), _stream()))

    def unique_experts(self, idx, expert_base, L, T, unique, total):
        _check(lib().unipool_unique_experts(self.handle, _p(idx), _p(expert_base), L, T, _p(unique), _p(total),
                                            _stream()))

    def profile_enable(self, on):
        _check(lib().unipool_profile_enable(self.handle, 1 if on else 0))

    def profile_read(self):
        """{phase name: (milliseconds, kernel launches)} since the last read."""
        n = len(PHASES)
        ms = (ctypes.c_double * n)()
        launches = (ctypes.c_int64 * n)()
        _check(lib().unipool_profile_read(self.handle, ms, launches))
        return {PHASES[i]: (float(ms[i]), int(launches[i])) for i in range(n)}

    def calibrate_c(self, n_experts, top_k, n_samples=100_000, seed=0):
        out = ctypes.c_float()
        _check(lib().unipool_calibrate_c(self.handle, n_experts, top_k, n_samples, seed, ctypes.byref(out),
                                         _stream()))
        return float(out.value)

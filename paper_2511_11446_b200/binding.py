"""ctypes binding of libdiffpro.so — argument marshalling only.

Every function has the name and argument order of its C entry point in ``include/diffpro.h``.
torch tensors supply device memory and the current CUDA stream; every step of the quantized
linear runs in the library's kernels. If the shared object is missing this module raises: there is
no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdiffpro.so")

DP_OK = 0
(DP_ERR_INVALID_ARG, DP_ERR_SHAPE, DP_ERR_ALIGN, DP_ERR_BITS, DP_ERR_WORKSPACE, DP_ERR_ARCH,
 DP_ERR_CUDA, DP_ERR_TIMEOUT) = range(1, 9)
DP_FLAG_NONE, DP_FLAG_FORCE_SIMT, DP_FLAG_FORCE_MMA, DP_FLAG_NO_PDL = 0, 1, 2, 4
DP_FLAG_CTA_PAIR, DP_FLAG_NO_CTA_PAIR = 0x800, 0x1000
DP_FLAG_WEIGHT_STATIONARY, DP_FLAG_NO_WEIGHT_STATIONARY = 0x2000, 0x4000
DP_FLAG_AUTOTUNE, DP_FLAG_GROUP_SMALL_M, DP_FLAG_FUSED_DAQ = 0x10000, 0x20000, 0x40000
DP_FLAG_UNPACK_FIRST, DP_FLAG_NO_UNPACK_FIRST = 0x80000, 0x100000
DP_FLAG_ACT_STATIONARY, DP_FLAG_NO_ACT_STATIONARY = 0x200000, 0x400000
DP_FLAG_TILE_N_MASK = 0x700
DP_PLAN_SAME_X, DP_PLAN_SAME_Y = 1, 2


def DP_FLAG_TILE_N(bn: int) -> int:
    return (bn // 64) << 8

DP_STATIC_SCRATCH_BYTES = 10 << 20

EXPORTS = ["dp_daq_quantize", "dp_daq_quantize_robust", "dp_wq_linear_workspace", "dp_wq_linear_workspace_grouped", "dp_wq_linear", "dp_wq_linear_static", "dp_wq_linear_residual", "dp_ln_modulate_daq", "dp_plan_create",
           "dp_plan_workspace", "dp_plan_layer_variant", "dp_plan_layer_unpack_first", "dp_plan_set_layer_flags", "dp_plan_set_daq", "dp_plan_destroy", "dp_plan_run", "dp_plan_x_bytes",
           "dp_plan_run_host", "dp_plan_phase_a", "dp_layer_latency_us", "dp_pack_weights_host", "dp_clip_rank", "dp_debug_skip_stage_load",
           "dp_status_string",
           "dp_last_error", "dp_version"]


class dp_weight(C.Structure):
    _fields_ = [("N", C.c_int32), ("K", C.c_int32), ("bits", C.c_int32), ("group_size", C.c_int32),
                ("qweight", C.c_void_p), ("s_w", C.c_void_p), ("bias", C.c_void_p), ("zeros", C.c_void_p)]


class dp_debug(C.Structure):
    _fields_ = [("q", C.c_void_p), ("ldq", C.c_int64), ("s_a", C.c_void_p), ("acc", C.c_void_p),
                ("ldacc", C.c_int64)]


class dp_phase_a_problem(C.Structure):
    _fields_ = [("n_steps", C.c_int32), ("drift", C.c_void_p), ("step_cost", C.c_void_p), ("n_layers", C.c_int32),
                ("n_options", C.c_void_p), ("opt_bits", C.c_void_p), ("opt_c_lat", C.c_void_p),
                ("opt_c_mem", C.c_void_p), ("sens", C.c_void_p), ("B_lat", C.c_double), ("B_mem", C.c_double),
                ("rho", C.c_double), ("eps", C.c_double)]


class DiffproError(RuntimeError):
    def __init__(self, status, where):
        self.status = status
        msg = lib().dp_last_error().decode()
        super().__init__(f"{where}: {lib().dp_status_string(status).decode()} ({msg})")


_lib = None


def lib():
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                               "`python -m paper_2511_11446_b200.build` (no fallback exists)")
        L = C.CDLL(LIB_PATH)
        L.dp_wq_linear_workspace.restype = C.c_size_t
        L.dp_wq_linear_workspace.argtypes = [C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_uint32]
        L.dp_wq_linear_workspace_grouped.restype = C.c_size_t
        L.dp_wq_linear_workspace_grouped.argtypes = [C.c_int64, C.POINTER(dp_weight)]
        L.dp_plan_workspace.restype = C.c_size_t
        L.dp_plan_workspace.argtypes = [C.c_void_p]
        L.dp_plan_layer_variant.argtypes = [C.c_void_p, C.c_int32] + [C.POINTER(C.c_int32)] * 4
        L.dp_plan_layer_unpack_first.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32)]
        L.dp_plan_set_layer_flags.argtypes = [C.c_void_p, C.c_int32, C.c_uint32]
        L.dp_plan_set_daq.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.POINTER(C.c_int32)]
        L.dp_plan_x_bytes.restype = C.c_size_t
        L.dp_plan_x_bytes.argtypes = [C.c_void_p]
        L.dp_plan_destroy.restype = None
        L.dp_plan_destroy.argtypes = [C.c_void_p]
        L.dp_status_string.restype = C.c_char_p
        L.dp_last_error.restype = C.c_char_p
        L.dp_daq_quantize_robust.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_int64,
                                             C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        L.dp_daq_quantize.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p,
                                      C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p]
        L.dp_wq_linear.argtypes = [C.POINTER(dp_weight), C.c_void_p, C.c_int64, C.c_void_p, C.c_int64,
                                   C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t,
                                   C.POINTER(dp_debug), C.c_void_p, C.c_uint32, C.c_void_p]
        L.dp_ln_modulate_daq.argtypes = [C.c_void_p, C.c_int64, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_int64,
                                         C.c_float, C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p]
        L.dp_wq_linear_residual.argtypes = [C.POINTER(dp_weight), C.c_void_p, C.c_int64, C.c_int64, C.POINTER(dp_residual),
                                            C.c_void_p, C.c_int64, C.c_void_p, C.c_size_t, C.c_void_p, C.c_uint32,
                                            C.c_void_p]
        L.dp_wq_linear_static.argtypes = [C.POINTER(dp_weight), C.c_void_p, C.c_int64, C.c_int64, C.c_void_p,
                                          C.c_int64, C.c_void_p, C.c_uint32, C.c_void_p]
        L.dp_plan_create.argtypes = [C.POINTER(dp_weight), C.c_int32, C.POINTER(C.c_int64), C.c_uint32,
                                     C.POINTER(C.c_void_p)]
        L.dp_plan_run.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_int32, C.c_int32,
                                  C.POINTER(C.c_void_p), C.POINTER(C.c_void_p), C.c_void_p, C.c_size_t,
                                  C.c_void_p, C.c_uint32, C.c_void_p]
        L.dp_plan_run_host.argtypes = [C.c_void_p, C.POINTER(C.c_int32), C.c_int32,
                                       C.POINTER(C.c_void_p), C.c_void_p, C.c_size_t,
                                       C.POINTER(C.c_void_p), C.c_int32, C.POINTER(C.c_void_p),
                                       C.c_void_p, C.c_size_t, C.c_void_p, C.c_uint32, C.c_void_p]
        L.dp_pack_weights_host.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_void_p]
        L.dp_plan_phase_a.argtypes = [C.POINTER(dp_phase_a_problem), C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.dp_layer_latency_us.argtypes = [C.POINTER(dp_weight), C.c_int64, C.c_uint32, C.c_int32, C.c_void_p]
        L.dp_clip_rank.restype = C.c_int32
        L.dp_clip_rank.argtypes = [C.c_int32, C.c_int32]
        L.dp_debug_skip_stage_load.restype = None
        L.dp_debug_skip_stage_load.argtypes = [C.c_int32]
        _lib = L
    return _lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _check(st, where):
    if st != DP_OK:
        raise DiffproError(st, where)


def make_weight(qweight: torch.Tensor, s_w: torch.Tensor, bias, N: int, K: int, bits: int, group_size: int = 0,
                zeros=None) -> dp_weight:
    return dp_weight(N, K, bits, group_size, qweight.data_ptr(), s_w.data_ptr(),
                     None if bias is None else bias.data_ptr(), None if zeros is None else zeros.data_ptr())


def dp_daq_quantize(x, M, K, ldx, q, ldq, s_a, rowsum=None, stream=None):
    _check(lib().dp_daq_quantize(_ptr(x), M, K, ldx, _ptr(q), ldq, _ptr(s_a), _ptr(rowsum),
                                 _stream(stream)), "dp_daq_quantize")


def dp_wq_linear_workspace(M, N, K, bits, flags=0) -> int:
    return int(lib().dp_wq_linear_workspace(M, N, K, bits, flags))


def dp_wq_linear_workspace_grouped(M, w: dp_weight) -> int:
    return int(lib().dp_wq_linear_workspace_grouped(M, C.byref(w)))


def dp_clip_rank(clip_percentile_e3: int, K: int) -> int:
    """The clip_rank dp_daq_quantize_robust takes for a percentile given in 1/1000 percent."""
    return int(lib().dp_clip_rank(clip_percentile_e3, K))


def dp_debug_skip_stage_load(k_block: int):
    lib().dp_debug_skip_stage_load(k_block)


def dp_daq_quantize_robust(x, M, K, ldx, q, ldq, s_a, rank, act_bits=8, rowsum=None, stream=None):
    _check(lib().dp_daq_quantize_robust(_ptr(x), M, K, ldx, _ptr(q), ldq, _ptr(s_a), _ptr(rowsum), rank, act_bits,
                                        _stream(stream)), "dp_daq_quantize_robust")


def dp_wq_linear(w: dp_weight, x, ldx, s_a_in, M, y, ldy, workspace, dbg: dp_debug | None = None,
                 device_status=None, flags=0, stream=None):
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().dp_wq_linear(C.byref(w), _ptr(x), ldx, _ptr(s_a_in), M, _ptr(y), ldy, _ptr(workspace),
                              ws_bytes, None if dbg is None else C.byref(dbg), _ptr(device_status),
                              flags, _stream(stream)), "dp_wq_linear")


def dp_ln_modulate_daq(x, M, K, ldx, shift, scale, rows_per_sample, eps, q, ldq, s_a, stream=None):
    """LayerNorm + adaLN modulation + DAQ of bf16 tokens in one pass (shift, scale may both be None)."""
    _check(lib().dp_ln_modulate_daq(_ptr(x), M, K, ldx, _ptr(shift), _ptr(scale), rows_per_sample, eps, _ptr(q), ldq,
                                    _ptr(s_a), _stream(stream)), "dp_ln_modulate_daq")


class dp_residual(C.Structure):
    _fields_ = [("residual", C.c_void_p), ("ldr", C.c_int64), ("gate", C.c_void_p), ("rows_per_gate", C.c_int64)]


def dp_wq_linear_residual(w: dp_weight, x, ldx, M, residual, ldr, gate, rows_per_gate, y, ldy, workspace, ws_bytes,
                          device_status=None, flags=0, stream=None):
    """dp_wq_linear on bf16 activations with y = bf16(gate * lin + residual) (gate None: lin + residual)
    in the epilogue; residual may be y."""
    r = dp_residual(residual.data_ptr(), ldr, None if gate is None else gate.data_ptr(), rows_per_gate)
    _check(lib().dp_wq_linear_residual(C.byref(w), _ptr(x), ldx, M, C.byref(r), _ptr(y), ldy, _ptr(workspace),
                                       ws_bytes, _ptr(device_status), flags, _stream(stream)), "dp_wq_linear_residual")


def dp_wq_linear_static(w: dp_weight, x, ldx, M, y, ldy, device_status=None, flags=0, stream=None):
    """dp_wq_linear without a workspace argument: the scratch is a fixed array inside the library
    (for callers that may not allocate device memory). bf16 input only."""
    _check(lib().dp_wq_linear_static(C.byref(w), _ptr(x), ldx, M, _ptr(y), ldy, _ptr(device_status), flags,
                                     _stream(stream)), "dp_wq_linear_static")


def dp_plan_create(weights: list[dp_weight], Ms: list[int], flags=0) -> C.c_void_p:
    arr = (dp_weight * len(weights))(*weights)
    ms = (C.c_int64 * len(Ms))(*Ms)
    out = C.c_void_p()
    _check(lib().dp_plan_create(arr, len(weights), ms, flags, C.byref(out)), "dp_plan_create")
    return out


def dp_plan_workspace(plan) -> int:
    return int(lib().dp_plan_workspace(plan))


def dp_plan_layer_variant(plan, layer: int) -> dict:
    """{'tile_n', 'cta_group', 'weight_stationary', 'small_m', 'unpack_first'} of one layer of a plan."""
    v = [C.c_int32() for _ in range(4)]
    _check(lib().dp_plan_layer_variant(plan, layer, *[C.byref(t) for t in v]), "dp_plan_layer_variant")
    u = C.c_int32(0)
    _check(lib().dp_plan_layer_unpack_first(plan, layer, C.byref(u)), "dp_plan_layer_unpack_first")
    return dict(tile_n=v[0].value, cta_group=v[1].value, weight_stationary=v[2].value, small_m=v[3].value,
                unpack_first=u.value)


def dp_plan_set_layer_flags(plan, layer: int, flags: int):
    _check(lib().dp_plan_set_layer_flags(plan, layer, flags), "dp_plan_set_layer_flags")


def dp_plan_set_daq(plan, clip_percentile_e3: int, n_timesteps: int = 0, act_bits_by_bin=None):
    bins = None if act_bits_by_bin is None else (C.c_int32 * 3)(*act_bits_by_bin)
    _check(lib().dp_plan_set_daq(plan, clip_percentile_e3, n_timesteps, bins), "dp_plan_set_daq")


def variant_flags(v: dict) -> int:
    """dp_wq_linear flags that force the kernel variant a plan chose for a layer."""
    if v["small_m"]:
        return DP_FLAG_FORCE_SIMT
    f = DP_FLAG_FORCE_MMA | DP_FLAG_TILE_N(v["tile_n"])
    f |= DP_FLAG_UNPACK_FIRST if v.get("unpack_first") else DP_FLAG_NO_UNPACK_FIRST
    if v["weight_stationary"] == 2:
        return f | DP_FLAG_ACT_STATIONARY
    if v["weight_stationary"]:
        return f | DP_FLAG_WEIGHT_STATIONARY
    f |= DP_FLAG_NO_WEIGHT_STATIONARY | DP_FLAG_NO_ACT_STATIONARY
    return f | (DP_FLAG_CTA_PAIR if v["cta_group"] == 2 else DP_FLAG_NO_CTA_PAIR)


def dp_plan_x_bytes(plan) -> int:
    return int(lib().dp_plan_x_bytes(plan))


def dp_plan_destroy(plan):
    lib().dp_plan_destroy(plan)


def ptr_array(ptrs):
    return (C.c_void_p * len(ptrs))(*ptrs)


def dp_plan_run(plan, steps, start_index, x_ptrs, y_ptrs, workspace, device_status=None, flags=0,
                stream=None):
    """x_ptrs / y_ptrs: ctypes arrays of device addresses (see ptr_array)."""
    st = (C.c_int32 * len(steps))(*steps)
    _check(lib().dp_plan_run(plan, st, len(steps), start_index, x_ptrs, y_ptrs, _ptr(workspace),
                             workspace.numel() * workspace.element_size(), _ptr(device_status), flags,
                             _stream(stream)), "dp_plan_run")


def dp_plan_run_host(plan, steps, x_host, x_stage, y_dev, d2h_layer, y_host, workspace,
                     device_status=None, flags=0, stream=None):
    st = (C.c_int32 * len(steps))(*steps)
    _check(lib().dp_plan_run_host(plan, st, len(steps), x_host, _ptr(x_stage),
                                  x_stage.numel() * x_stage.element_size(), y_dev, d2h_layer, y_host,
                                  _ptr(workspace), workspace.numel() * workspace.element_size(),
                                  _ptr(device_status), flags, _stream(stream)), "dp_plan_run_host")


def dp_plan_phase_a(drift, step_cost, options, sens, B_lat, B_mem, rho, eps):
    """options[l] = list of (bits, c_lat, c_mem), largest bits first; the arrays are host data.
    Returns (bitplan list, kept list of 0/1, (C_lat, C_mem), feasible)."""
    import numpy as np
    T, nl = len(drift), len(options)
    d = np.ascontiguousarray(drift, np.float64)
    c = np.ascontiguousarray(step_cost, np.float64)
    n_opt = np.array([len(o) for o in options], np.int32)
    bits = np.array([b for o in options for (b, _, _) in o], np.int32)
    lat = np.array([x for o in options for (_, x, _) in o], np.float64)
    mem = np.array([x for o in options for (_, _, x) in o], np.float64)
    s = np.ascontiguousarray(sens, np.float64)
    p = lambda a: a.ctypes.data_as(C.c_void_p)
    prob = dp_phase_a_problem(T, p(d), p(c), nl, p(n_opt), p(bits), p(lat), p(mem), p(s), B_lat, B_mem, rho, eps)
    plan, kept, tot, ok = np.empty(nl, np.int32), np.empty(T, np.uint8), np.empty(2, np.float64), C.c_int32(0)
    _check(lib().dp_plan_phase_a(C.byref(prob), p(plan), p(kept), p(tot), C.byref(ok)), "dp_plan_phase_a")
    return plan.tolist(), kept.tolist(), (float(tot[0]), float(tot[1])), bool(ok.value)


def dp_layer_latency_us(w: dp_weight, M: int, flags=0, reps=20) -> float:
    us = C.c_float(0.0)
    _check(lib().dp_layer_latency_us(C.byref(w), M, flags, reps, C.byref(us)), "dp_layer_latency_us")
    return float(us.value)


def dp_pack_weights_host(w, bits: int):
    """w: numpy int8 [N,K] -> numpy packed array (int8 [N,K] or uint32 [N, K*bits/32])."""
    import numpy as np
    assert w.dtype == np.int8 and w.flags.c_contiguous
    N, K = w.shape
    out = np.empty((N, K), np.int8) if bits == 8 else np.empty((N, K * bits // 32), np.uint32)
    _check(lib().dp_pack_weights_host(w.ctypes.data_as(C.c_void_p), N, K, bits,
                                      out.ctypes.data_as(C.c_void_p)), "dp_pack_weights_host")
    return out


def dp_version() -> int:
    return int(lib().dp_version())

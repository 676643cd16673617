"""CPU oracle of the DiffPro quantized linear — TEST INFRASTRUCTURE ONLY.

numpy-facing wrappers around ``diffpro_oracle.c`` (plain C, fp32/int arithmetic exactly as the
definitions state). Only the tests, the smoke check and the benchmark's cpu-baseline leg may import
this package; the CUDA library never does, and this package never imports the CUDA library.

bf16 tensors are carried as ``numpy.uint16`` bit patterns.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "diffpro_oracle.c")
_LIB = os.path.join(_HERE, "libdiffpro_oracle.so")
CFLAGS = ["-O2", "-fno-fast-math", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc if the shared object is missing or older than its source."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        subprocess.check_call(["gcc", *CFLAGS, "-o", _LIB, _SRC, "-lm"])
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.orc_num_threads.restype = C.c_int
        _lib.orc_pack.restype = C.c_int64
        _lib.orc_bf16_to_f32.restype = C.c_float
        _lib.orc_bf16_to_f32.argtypes = [C.c_uint16]
        _lib.orc_f32_to_bf16.restype = C.c_uint16
        _lib.orc_f32_to_bf16.argtypes = [C.c_float]
    return _lib


def num_threads() -> int:
    return int(lib().orc_num_threads())


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _i64(v):
    return C.c_int64(int(v))


def _chk(a, dtype, name):
    assert a.dtype == dtype and a.flags.c_contiguous, f"{name}: need contiguous {dtype}"


def row_words(K: int, bits: int) -> int:
    return (K * bits + 31) // 32


def daq(x: np.ndarray):
    """x: uint16 (bf16 bits) [M, K] -> (q int8 [M,K], s_a fp32 [M], rowsum int32 [M])."""
    _chk(x, np.uint16, "x")
    M, K = x.shape
    q = np.empty((M, K), np.int8)
    s_a = np.empty(M, np.float32)
    rowsum = np.empty(M, np.int32)
    lib().orc_daq(_p(x), _i64(M), _i64(K), _i64(K), _p(q), _i64(K), _p(s_a), _p(rowsum))
    return q, s_a, rowsum


def clip_rank(p, K: int) -> int:
    """Rank from the top of the nearest-rank p-th percentile of K values (p = 100 -> 1): the
    ceil(p K / 100)-th smallest is the (K - ceil(p K / 100) + 1)-th largest. p may be a str/Fraction."""
    from fractions import Fraction
    import math
    f = Fraction(str(p)) * K / 100
    return K - max(1, math.ceil(f)) + 1


def daq_robust(x: np.ndarray, rank: int, act_bits: int = 8):
    """Eq. "daq" with the clip threshold at the rank-th largest magnitude of each token and
    act_bits-bit codes: x uint16 (bf16 bits) [M, K] -> (q int8, s_a fp32 [M], rowsum int32 [M])."""
    _chk(x, np.uint16, "x")
    M, K = x.shape
    q = np.empty((M, K), np.int8)
    s_a = np.empty(M, np.float32)
    rowsum = np.empty(M, np.int32)
    st = lib().orc_daq_robust(_p(x), _i64(M), _i64(K), _i64(K), C.c_int(rank), C.c_int(act_bits), _p(q), _i64(K),
                              _p(s_a), _p(rowsum))
    if st != 0:
        raise ValueError(f"bad clip rank {rank} (K = {K}) or activation bits {act_bits}")
    return q, s_a, rowsum


def pack(w: np.ndarray, bits: int) -> np.ndarray:
    """w int8 [N,K] -> packed: int8 [N,K] (bits 8) or uint32 [N, K*bits/32]."""
    _chk(w, np.int8, "w")
    N, K = w.shape
    out = np.empty((N, K), np.int8) if bits == 8 else np.empty((N, row_words(K, bits)), np.uint32)
    bad = lib().orc_pack(_p(w), _i64(N), _i64(K), C.c_int(bits), _p(out))
    if bad:
        raise ValueError(f"weight value out of range for {bits} bits at flat index {bad - 1}")
    return out


def unpack(packed: np.ndarray, K: int, bits: int) -> np.ndarray:
    assert packed.flags.c_contiguous
    N = packed.shape[0]
    w = np.empty((N, K), np.int8)
    lib().orc_unpack(_p(packed), _i64(N), _i64(K), C.c_int(bits), _p(w))
    return w


def gemm_i32(q: np.ndarray, w: np.ndarray) -> np.ndarray:
    _chk(q, np.int8, "q")
    _chk(w, np.int8, "w")
    M, K = q.shape
    N = w.shape[0]
    assert w.shape[1] == K
    acc = np.empty((M, N), np.int32)
    lib().orc_gemm_i32(_p(q), _i64(K), _p(w), _i64(M), _i64(N), _i64(K), _p(acc), _i64(N))
    return acc


def epilogue(acc, s_a, s_w, bias=None) -> np.ndarray:
    _chk(acc, np.int32, "acc")
    _chk(s_a, np.float32, "s_a")
    _chk(s_w, np.float32, "s_w")
    if bias is not None:
        _chk(bias, np.uint16, "bias")
    M, N = acc.shape
    y = np.empty((M, N), np.uint16)
    lib().orc_epilogue(_p(acc), _i64(N), _p(s_a), _p(s_w), _p(bias), _i64(M), _i64(N), _p(y),
                       _i64(N))
    return y


def wq_linear(x, qweight, s_w, bias, bits: int, taps: bool = False):
    """Full layer. Returns y (uint16 bf16 bits) and, with taps, (y, q, s_a, acc)."""
    _chk(x, np.uint16, "x")
    M, K = x.shape
    N = qweight.shape[0]
    if taps:
        q, s_a, _ = daq(x)
        w = unpack(qweight, K, bits)
        acc = gemm_i32(q, w)
        return epilogue(acc, s_a, s_w, bias), q, s_a, acc
    y = np.empty((M, N), np.uint16)
    sw_ = np.empty((N, K), np.int8)
    sq = np.empty((M, K), np.int8)
    ssa = np.empty(M, np.float32)
    sacc = np.empty((M, N), np.int32)
    lib().orc_wq_linear(_p(x), _i64(K), _i64(M), _i64(N), _i64(K), C.c_int(bits), _p(qweight),
                        _p(s_w), _p(bias), _p(y), _i64(N), _p(sw_), _p(sq), _p(ssa), _p(sacc))
    return y


def wq_linear_points(x, qweight, s_w, bias, bits: int, pm, pn):
    """Selected (m, n) outputs: returns (acc int32 [P], y uint16 [P])."""
    _chk(x, np.uint16, "x")
    M, K = x.shape
    N = qweight.shape[0]
    pm = np.ascontiguousarray(pm, np.int64)
    pn = np.ascontiguousarray(pn, np.int64)
    assert pm.shape == pn.shape and pm.max(initial=0) < M and pn.max(initial=0) < N
    acc = np.empty(pm.shape[0], np.int32)
    y = np.empty(pm.shape[0], np.uint16)
    lib().orc_wq_linear_points(_p(x), _i64(K), _i64(N), _i64(K), C.c_int(bits), _p(qweight),
                               _p(s_w), _p(bias), _p(pm), _p(pn), _i64(pm.shape[0]), _p(acc), _p(y))
    return acc, y


class _Layer(C.Structure):
    _fields_ = [("M", C.c_int64), ("N", C.c_int64), ("K", C.c_int64), ("bits", C.c_int32),
                ("qweight", C.c_void_p), ("s_w", C.c_void_p), ("bias", C.c_void_p)]


def plan_run(layers, kept, xs):
    """Algorithm 2 Phase B over the linears.

    layers: list of dicts {M,N,K,bits,qweight,s_w,bias}; kept: ascending retained timesteps;
    xs[i][l]: uint16 [M_l,K_l] input of layer l at kept[i]. Returns ys[i][l] (uint16 [M_l,N_l]).
    """
    nL, nS = len(layers), len(kept)
    arr = (_Layer * nL)()
    for l, L in enumerate(layers):
        arr[l] = _Layer(L["M"], L["N"], L["K"], L["bits"], _p(L["qweight"]).value,
                        _p(L["s_w"]).value, None if L["bias"] is None else _p(L["bias"]).value)
    ys = [[np.empty((L["M"], L["N"]), np.uint16) for L in layers] for _ in range(nS)]
    xp = (C.c_void_p * (nL * nS))(*[_p(xs[i][l]).value for i in range(nS) for l in range(nL)])
    yp = (C.c_void_p * (nL * nS))(*[_p(ys[i][l]).value for i in range(nS) for l in range(nL)])
    mx = lambda f: max(f(L) for L in layers)
    sw_ = np.empty(mx(lambda L: L["N"] * L["K"]), np.int8)
    sq = np.empty(mx(lambda L: L["M"] * L["K"]), np.int8)
    ssa = np.empty(mx(lambda L: L["M"]), np.float32)
    sacc = np.empty(mx(lambda L: L["M"] * L["N"]), np.int32)
    k = np.ascontiguousarray(kept, np.int32)
    lib().orc_plan_run(arr, C.c_int32(nL), _p(k), C.c_int32(nS), xp, yp, _p(sw_), _p(sq), _p(ssa),
                       _p(sacc))
    return ys


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns (uint16) to float32."""
    return (bits.astype(np.uint32) << 16).view(np.float32)


def phase_a(drift, step_cost, options, sens, B_lat, B_mem, rho, eps):
    """Algorithm 2, Phase A. options[l] = list of (bits, c_lat, c_mem), largest bits first.
    Returns (bitplan list, kept list of 0/1, (C_lat, C_mem), feasible)."""
    T, L = len(drift), len(options)
    d = np.ascontiguousarray(drift, np.float64)
    c = np.ascontiguousarray(step_cost, np.float64)
    n_opt = np.array([len(o) for o in options], np.int32)
    bits = np.array([b for o in options for (b, _, _) in o], np.int32)
    lat = np.array([x for o in options for (_, x, _) in o], np.float64)
    mem = np.array([x for o in options for (_, _, x) in o], np.float64)
    s = np.ascontiguousarray(sens, np.float64)
    plan = np.empty(L, np.int32)
    kept = np.empty(T, np.uint8)
    tot = np.empty(2, np.float64)
    f = lib().orc_phase_a
    f.restype = C.c_int
    f.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p,
                  C.c_void_p, C.c_double, C.c_double, C.c_double, C.c_double, C.c_void_p, C.c_void_p, C.c_void_p]
    ok = f(T, _p(d), _p(c), L, _p(n_opt), _p(bits), _p(lat), _p(mem), _p(s), B_lat, B_mem, rho, eps, _p(plan),
           _p(kept), _p(tot))
    return plan.tolist(), kept.tolist(), (float(tot[0]), float(tot[1])), bool(ok)


def linear_bf16(x, w, bias=None):
    """Pass-through linear of a 16-bit layer: x uint16 (bf16 bits) [M,K], w uint16 [N,K], bias uint16 [N]
    or None. Returns (y uint16 [M,N], exact float64 [M,N], mag float64 [M,N] = sum_k |x w|)."""
    _chk(x, np.uint16, "x")
    _chk(w, np.uint16, "w")
    M, K = x.shape
    N = w.shape[0]
    assert w.shape[1] == K
    y = np.empty((M, N), np.uint16)
    exact = np.empty((M, N), np.float64)
    mag = np.empty((M, N), np.float64)
    lib().orc_linear_bf16(_p(x), _i64(K), _p(w), _p(bias), _i64(M), _i64(N), _i64(K), _p(y), _i64(N), _p(exact),
                          _p(mag))
    return y, exact, mag


def wq_linear_grouped(x, qweight, s_w, bias, bits: int, g: int, zeros=None):
    """Layer with group-wise weight scales: s_w fp32 [N, K/g], zeros uint8 [N, K/g] or None (symmetric).
    Returns y uint16 [M, N]."""
    _chk(x, np.uint16, "x")
    _chk(s_w, np.float32, "s_w")
    M, K = x.shape
    N = qweight.shape[0]
    assert K % g == 0 and s_w.shape == (N, K // g)
    if zeros is not None:
        _chk(zeros, np.uint8, "zeros")
        assert zeros.shape == (N, K // g)
    y = np.empty((M, N), np.uint16)
    sw_ = np.empty((N, K), np.int8)
    sq = np.empty((M, K), np.int8)
    ssa = np.empty(M, np.float32)
    lib().orc_wq_linear_grouped(_p(x), _i64(K), _i64(M), _i64(N), _i64(K), C.c_int(bits), _i64(g), _p(qweight),
                                _p(s_w), _p(zeros), _p(bias), _p(y), _i64(N), _p(sw_), _p(sq), _p(ssa))
    return y


def wq_linear_residual(x, qweight, s_w, bias, bits: int, res, gate=None, rows_per_gate: int = 1):
    """Layer with the residual (and optional per-sample gate) taken into the epilogue. res uint16 [M, N];
    gate uint16 [ceil(M / rows_per_gate), N] or None. Returns y uint16 [M, N]."""
    _chk(x, np.uint16, "x")
    _chk(res, np.uint16, "res")
    M, K = x.shape
    N = qweight.shape[0]
    assert res.shape == (M, N)
    if gate is not None:
        _chk(gate, np.uint16, "gate")
        assert gate.shape == (-(-M // rows_per_gate), N)
    y = np.empty((M, N), np.uint16)
    sw_ = np.empty((N, K), np.int8)
    sq = np.empty((M, K), np.int8)
    ssa = np.empty(M, np.float32)
    sacc = np.empty((M, N), np.int32)
    lib().orc_wq_linear_residual(_p(x), _i64(K), _i64(M), _i64(N), _i64(K), C.c_int(bits), _p(qweight), _p(s_w),
                                 _p(bias), _p(res), _i64(N), _p(gate), _i64(rows_per_gate), _p(y), _i64(N), _p(sw_),
                                 _p(sq), _p(ssa), _p(sacc))
    return y


def ln_modulate_daq(x, shift=None, scale=None, rows_per_sample: int = 1, eps: float = 1e-6, tap=False):
    """LayerNorm (no affine) + adaLN modulation + DAQ of bf16 tokens x uint16 [M, K]; shift, scale uint16
    [ceil(M / rows_per_sample), K] or both None. Returns (q int8 [M,K], s_a fp32 [M]) and, with tap,
    the fp32 activations that were quantized."""
    _chk(x, np.uint16, "x")
    M, K = x.shape
    assert (shift is None) == (scale is None)
    if shift is not None:
        _chk(shift, np.uint16, "shift")
        _chk(scale, np.uint16, "scale")
        assert shift.shape == scale.shape == (-(-M // rows_per_sample), K)
    q = np.empty((M, K), np.int8)
    s_a = np.empty(M, np.float32)
    h = np.empty((M, K), np.float32) if tap else None
    lib().orc_ln_modulate_daq(_p(x), _i64(M), _i64(K), _i64(K), _p(shift), _p(scale), _i64(rows_per_sample),
                              C.c_float(eps), _p(q), _i64(K), _p(s_a), _p(h))
    return (q, s_a, h) if tap else (q, s_a)

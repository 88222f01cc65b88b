"""CPU oracle for the Q-ASR integer-only inference path -- TEST INFRASTRUCTURE ONLY.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It never imports the GPU package and shares no code with it.

The arithmetic lives in ``qasr_oracle.c`` (plain C loops, int64 intermediates);
this module compiles it with gcc on first use, wraps it with ctypes + numpy and
walks a model description layer by layer, keeping every intermediate tensor.

Passages followed: Sec. 2.1 Eq. 1 (integer grid, DQ), Sec. 2.2 (integer
convolution by linearity, integer ReLU, BatchNorm folded into the preceding
convolution).  The dyadic requantisation and the integer residual add are not
printed in the paper; the readings are stated in ``qasr_oracle.c``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qasr_oracle.c")
_LIB_PATH = os.path.join(_HERE, "libqasr_oracle.so")
_lock = threading.Lock()
_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O3 -fopenmp).  Returns the .so path."""
    with _lock:
        stale = (not os.path.exists(_LIB_PATH)
                 or os.path.getmtime(_LIB_PATH) < os.path.getmtime(_SRC))
        if force or stale:
            tmp = _LIB_PATH + ".tmp.%d" % os.getpid()
            cmd = ["gcc", "-O3", "-fopenmp", "-fPIC", "-shared", "-std=c11",
                   "-fno-fast-math", "-o", tmp, _SRC]
            subprocess.run(cmd, check=True)
            os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    if _lib is None:
        path = build()
        L = ctypes.CDLL(path)
        i8p = ctypes.POINTER(ctypes.c_int8)
        i32p = ctypes.POINTER(ctypes.c_int32)
        u8p = ctypes.POINTER(ctypes.c_uint8)
        f32p = ctypes.POINTER(ctypes.c_float)
        c_int = ctypes.c_int
        L.qo_num_threads.restype = c_int
        L.qo_rs.restype = ctypes.c_int64
        L.qo_rs.argtypes = [ctypes.c_int64, c_int]
        L.qo_sat8.restype = ctypes.c_int64
        L.qo_sat8.argtypes = [ctypes.c_int64]
        L.qo_conv1d.restype = c_int
        L.qo_conv1d.argtypes = [i8p, c_int, c_int, c_int, i8p, c_int, c_int, c_int, c_int, c_int, i32p, i32p]
        L.qo_requant.restype = c_int
        L.qo_requant.argtypes = [i32p, c_int, c_int, c_int, i32p, u8p, c_int, i8p]
        L.qo_residual_add.restype = c_int
        L.qo_residual_add.argtypes = [c_int, ctypes.POINTER(i8p), i32p, u8p, ctypes.c_size_t, c_int, i8p]
        L.qo_dequant.restype = c_int
        L.qo_dequant.argtypes = [i32p, c_int, c_int, c_int, f32p, f32p]
        L.qo_glu.restype = c_int
        L.qo_glu.argtypes = [i8p, i8p, c_int, c_int, c_int, c_int, i32p, u8p, i8p]
        _lib = L
    return _lib


def num_threads() -> int:
    return int(lib().qo_num_threads())


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct))


def _c(a, dtype):
    a = np.ascontiguousarray(a, dtype=dtype)
    return a


def _check(rc, what):
    if rc != 0:
        raise RuntimeError("oracle %s failed with code %d" % (what, rc))


# ----------------------------------------------------------------------------- scalars
def rs(v: int, c: int) -> int:
    """RS(v, c) = floor((v + 2^(c-1)) / 2^c) on a 64-bit signed value."""
    return int(lib().qo_rs(int(v), int(c)))


def sat8(v: int) -> int:
    return int(lib().qo_sat8(int(v)))


# ----------------------------------------------------------------------------- tensors
def out_len(T: int, stride: int) -> int:
    return (T - 1) // stride + 1


def conv1d(x, w, bias=None, stride=1, dilation=1, depthwise=False):
    """Integer conv (Sec. 2.2): x int8 [B][C_in][T]; w int8 [C_out][C_in][K] (or
    [C][K] when depthwise) -> int32 accumulator [B][C_out][T_out] (bias added)."""
    x = _c(x, np.int8)
    w = _c(w, np.int8)
    B, C_in, T = x.shape
    if depthwise:
        C_out, K = w.shape
    else:
        if w.ndim == 2:
            w = w[:, :, None]
        C_out, ci, K = w.shape
        assert ci == C_in, (ci, C_in)
        w = np.ascontiguousarray(w)
    T_out = out_len(T, stride)
    acc = np.empty((B, C_out, T_out), dtype=np.int32)
    bptr = None
    if bias is not None:
        bias = _c(bias, np.int32)
        assert bias.shape == (C_out,)
        bptr = _p(bias, ctypes.c_int32)
    rc = lib().qo_conv1d(_p(x, ctypes.c_int8), B, C_in, T, _p(w, ctypes.c_int8), C_out, K,
                         stride, dilation, 1 if depthwise else 0, bptr, _p(acc, ctypes.c_int32))
    _check(rc, "conv1d")
    return acc


def requant(acc, mult, shift, relu=False):
    """Per-channel dyadic requantisation of an int32 accumulator to int8."""
    acc = _c(acc, np.int32)
    B, C, T = acc.shape
    mult = _c(mult, np.int32)
    shift = _c(shift, np.uint8)
    assert mult.shape == (C,) and shift.shape == (C,)
    y = np.empty((B, C, T), dtype=np.int8)
    rc = lib().qo_requant(_p(acc, ctypes.c_int32), B, C, T, _p(mult, ctypes.c_int32),
                          _p(shift, ctypes.c_uint8), 1 if relu else 0, _p(y, ctypes.c_int8))
    _check(rc, "requant")
    return y


def residual_add(terms, mult, shift, relu=False):
    """Integer residual add: per-term dyadic rescale (rounded per term), sum, ReLU, clamp."""
    terms = [_c(t, np.int8) for t in terms]
    shape = terms[0].shape
    for t in terms:
        assert t.shape == shape
    mult = _c(mult, np.int32)
    shift = _c(shift, np.uint8)
    assert mult.shape == (len(terms),) and shift.shape == (len(terms),)
    i8p = ctypes.POINTER(ctypes.c_int8)
    arr = (i8p * len(terms))(*[_p(t, ctypes.c_int8) for t in terms])
    y = np.empty(shape, dtype=np.int8)
    rc = lib().qo_residual_add(len(terms), arr, _p(mult, ctypes.c_int32), _p(shift, ctypes.c_uint8),
                               terms[0].size, 1 if relu else 0, _p(y, ctypes.c_int8))
    _check(rc, "residual_add")
    return y


def dequant(acc, scale):
    """DQ (Eq. 1's inverse) of the last layer's int32 output, one fp32 multiply each."""
    acc = _c(acc, np.int32)
    B, C, T = acc.shape
    scale = _c(scale, np.float32)
    assert scale.shape == (C,)
    out = np.empty((B, C, T), dtype=np.float32)
    rc = lib().qo_dequant(_p(acc, ctypes.c_int32), B, C, T, _p(scale, ctypes.c_float), _p(out, ctypes.c_float))
    _check(rc, "dequant")
    return out


def glu(a, q, q_c, mult, shift):
    a = _c(a, np.int8)
    q = _c(q, np.int8)
    B, C, T = a.shape
    mult = _c(mult, np.int32)
    shift = _c(shift, np.uint8)
    y = np.empty((B, C, T), dtype=np.int8)
    rc = lib().qo_glu(_p(a, ctypes.c_int8), _p(q, ctypes.c_int8), B, C, T, int(q_c),
                      _p(mult, ctypes.c_int32), _p(shift, ctypes.c_uint8), _p(y, ctypes.c_int8))
    _check(rc, "glu")
    return y


# ----------------------------------------------------------------------------- host helpers
def quantize(x, S):
    """Eq. 1 with b = 8: q = clamp(Int(x / S)) to [-128, 127]; Int = round half away from zero."""
    r = np.asarray(x, dtype=np.float64) / float(S)
    q = np.sign(r) * np.floor(np.abs(r) + 0.5)
    return np.clip(q, -128, 127).astype(np.int8)


def fold_batchnorm(W, gamma, beta, mean, var, eps):
    """BatchNorm folded into the preceding conv (Sec. 2.2): returns (W', b') in float64 with
    conv(W', x) + b' == BN(conv(W, x))."""
    W = np.asarray(W, dtype=np.float64)
    g = np.asarray(gamma, np.float64) / np.sqrt(np.asarray(var, np.float64) + eps)
    Wf = W * g.reshape((-1,) + (1,) * (W.ndim - 1))
    bf = np.asarray(beta, np.float64) - np.asarray(mean, np.float64) * g
    return Wf, bf


def dyadic_encode(M: float, lo_bits: int = 14):
    """Encode a positive real multiplier as mult / 2^shift with mult in [2^lo_bits, 2^(lo_bits+1))."""
    assert M > 0
    shift = 0
    m = M
    while m < (1 << lo_bits):
        m *= 2.0
        shift += 1
    while m >= (1 << (lo_bits + 1)):
        m /= 2.0
        shift -= 1
    mult = int(np.floor(m + 0.5))
    if mult == (1 << (lo_bits + 1)):
        mult //= 2
        shift -= 1
    assert 1 <= shift <= 62, shift
    return mult, shift


# ----------------------------------------------------------------------------- layer and model walk
def run_layer(layer, bufs):
    """Run one entry of a model description (see workloads/) on the buffer dict ``bufs``.
    Returns a dict of every tensor the layer produced (by role)."""
    kind = layer["kind"]
    out = {}
    if kind == "add":
        terms = [bufs[i] for i in layer["res"]]
        y = residual_add(terms, layer["res_m"], layer["res_s"], relu=layer["relu"])
        out["y"] = y
        bufs[layer["out"]] = y
        return out
    x = bufs[layer["in"]]
    if kind == "glu":
        C = layer["C_out"]
        y = glu(x[:, :C, :], x[:, C:, :], layer["q_c"], layer["m"], layer["s"])
        out["y"] = y
        bufs[layer["out"]] = y
        return out
    if kind in ("tcs", "dw"):
        acc_dw = conv1d(x, layer["w_dw"], None, layer["stride"], layer["dilation"], depthwise=True)
        h = requant(acc_dw, layer["m_dw"], layer["s_dw"], relu=False)
        out["dw"] = h
        if kind == "dw":
            out["y"] = h
            bufs[layer["out"]] = h
            return out
        acc = conv1d(h, layer["w"], layer.get("bias"), 1, 1, depthwise=False)
    elif kind == "pw":
        acc = conv1d(x, layer["w"], layer.get("bias"), 1, 1, depthwise=False)
    elif kind == "dense":
        acc = conv1d(x, layer["w"], layer.get("bias"), layer["stride"], layer["dilation"], depthwise=False)
    else:
        raise ValueError("unknown layer kind %r" % (kind,))
    if layer.get("out_int32"):
        out["y"] = acc
        bufs[layer["out"]] = acc
        return out
    res = layer.get("res") or []
    if res:
        # main branch: requant and clamp to int8 first (no ReLU), then the integer residual add
        a = requant(acc, layer["m"], layer["s"], relu=False)
        out["main"] = a
        terms = [a] + [bufs[i] for i in res]
        y = residual_add(terms, layer["res_m"], layer["res_s"], relu=layer["relu"])
    else:
        y = requant(acc, layer["m"], layer["s"], relu=layer["relu"])
    out["y"] = y
    bufs[layer["out"]] = y
    return out


def encoder_forward(model, x, keep=True):
    """Forward pass over a model description.  Returns (logits_q int32, logits float32, trace)
    where trace[i] is the dict of tensors layer i produced (empty dicts if keep is False)."""
    bufs = {0: _c(x, np.int8)}
    trace = []
    last = None
    for layer in model["layers"]:
        o = run_layer(layer, bufs)
        last = o["y"]
        trace.append(o if keep else {})
    assert last.dtype == np.int32, "the last layer must leave int32 logits"
    logits = dequant(last, model["out_scale"])
    return last, logits, trace

"""ctypes binding of libqasr.so: the same entry points as include/qasr.h, argument
marshalling only.  Tensors are torch CUDA tensors (used for device memory and streams);
every arithmetic step runs inside the library's kernels."""
from __future__ import annotations

import ctypes
import os

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
MAX_TERMS = 12
OPT_GRAPH, OPT_TENSOR_CORES, OPT_PROFILE, OPT_STATIC_WEIGHTS = 1, 2, 4, 5
OPT_GEMM_FRAME_TILE, OPT_DW_FRAME_TILE, OPT_SIDE_BRANCH, OPT_FRAME_MAJOR_OUTPUT = 6, 7, 8, 9
LAYER_KINDS = {"dw": 1, "pw": 2, "dense": 3, "tcs": 4, "add": 5, "glu": 6}


def lib_path() -> str:
    return os.path.join(_HERE, "libqasr.so")


class QasrError(RuntimeError):
    def __init__(self, code, text, detail=""):
        super().__init__("qasr error %d (%s)%s" % (code, text, (": " + detail) if detail else ""))
        self.code = code


class QasrRequant(ctypes.Structure):
    _fields_ = [("mult", ctypes.c_void_p), ("shift", ctypes.c_void_p)]


class QasrLayer(ctypes.Structure):
    _fields_ = [
        ("kind", ctypes.c_int32), ("in_buf", ctypes.c_int32), ("out_buf", ctypes.c_int32),
        ("C_in", ctypes.c_int32), ("C_out", ctypes.c_int32),
        ("K", ctypes.c_int32), ("stride", ctypes.c_int32), ("dilation", ctypes.c_int32),
        ("w_dw", ctypes.c_void_p), ("rq_dw", QasrRequant),
        ("w", ctypes.c_void_p), ("bias", ctypes.c_void_p), ("max_abs_bias", ctypes.c_int32),
        ("rq", QasrRequant),
        ("relu", ctypes.c_int32), ("out_int32", ctypes.c_int32), ("glu_qc", ctypes.c_int32),
        ("n_terms", ctypes.c_int32),
        ("term_buf", ctypes.c_int32 * MAX_TERMS), ("term_mult", ctypes.c_int32 * MAX_TERMS),
        ("term_shift", ctypes.c_uint8 * MAX_TERMS),
    ]


class QasrProfileEntry(ctypes.Structure):
    _fields_ = [("layer", ctypes.c_int32), ("kernel", ctypes.c_int32), ("ms", ctypes.c_float),
                ("reserved", ctypes.c_float), ("macs", ctypes.c_double), ("bytes", ctypes.c_double)]


_lib = None


def lib():
    """Loads libqasr.so; raises ImportError if it has not been built (no fallback exists)."""
    global _lib
    if _lib is not None:
        return _lib
    path = lib_path()
    if not os.path.exists(path):
        raise ImportError("%s is missing: build it with `python -m paper_2103_16827_b200.build`" % path)
    L = ctypes.CDLL(path)
    vp, ci, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    P = ctypes.POINTER
    L.qasr_create.argtypes = [P(vp), ci, vp]
    L.qasr_destroy.argtypes = [vp]
    L.qasr_strerror.argtypes = [ci]
    L.qasr_strerror.restype = ctypes.c_char_p
    L.qasr_last_error.argtypes = [vp]
    L.qasr_last_error.restype = ctypes.c_char_p
    L.qasr_poll_status.argtypes = [vp]
    L.qasr_set_option.argtypes = [vp, ci, ci]
    L.qasr_selftest_wait_timeout.argtypes = [vp, ctypes.c_uint]
    L.qasr_selftest_wait_timeout.restype = ci
    L.qasr_measure_int8_tensor_peak.argtypes = [vp, ci, P(ctypes.c_float), P(ctypes.c_double)]
    L.qasr_measure_int8_tensor_peak.restype = ci
    L.qasr_launch_count.argtypes = [vp]
    L.qasr_launch_count.restype = ctypes.c_int64
    L.qasr_dw_conv.argtypes = [vp, vp, ci, ci, ci, vp, ci, ci, ci, QasrRequant, vp]
    L.qasr_conv.argtypes = [vp, vp, ci, ci, ci, vp, ci, ci, ci, ci, vp, ctypes.c_int32, QasrRequant, ci,
                            ci, P(vp), P(ctypes.c_int32), P(ctypes.c_uint8), vp, vp]
    L.qasr_conv_scratch_bytes.argtypes = [ci, ci, ci, ci, ci, ci, P(cs)]
    L.qasr_set_conv_scratch.argtypes = [vp, vp, cs]
    L.qasr_tcs_block_workspace_bytes.argtypes = [ci, ci, ci, ci, ci, ci, ci, P(cs)]
    L.qasr_tcs_block.argtypes = [vp, vp, ci, ci, ci, vp, ci, ci, ci, QasrRequant, vp, ci, vp, ctypes.c_int32,
                                 QasrRequant, ci, vp, vp, cs]
    L.qasr_tcs_block_noalloc.argtypes = [ci, vp, vp, ci, ci, ci, vp, ci, ci, ci, QasrRequant, vp, ci, vp, ctypes.c_int32,
                                         QasrRequant, ci, vp, ci]
    L.qasr_tcs_block_noalloc.restype = ci
    L.qasr_residual_requant_add.argtypes = [vp, ci, P(vp), P(ctypes.c_int32), P(ctypes.c_uint8), ci, ci, ci, ci, vp]
    L.qasr_dequant_logits.argtypes = [vp, vp, ci, ci, ci, vp, vp]
    L.qasr_glu.argtypes = [vp, vp, ci, ci, ci, ci, QasrRequant, vp]
    L.qasr_glu.restype = ci
    L.qasr_encoder_workspace_bytes.argtypes = [P(QasrLayer), ci, ci, ci, ci, P(cs)]
    L.qasr_encoder_forward.argtypes = [vp, P(QasrLayer), ci, vp, ci, ci, ci, vp, cs, vp, vp, vp]
    L.qasr_encoder_buffer_info.argtypes = [P(QasrLayer), ci, ci, ci, ci, ci, P(cs), P(ci), P(ci)]
    L.qasr_encoder_host_staging_bytes.argtypes = [P(QasrLayer), ci, ci, ci, ci, P(cs)]
    L.qasr_encoder_forward_host.argtypes = [vp, P(QasrLayer), ci, vp, ci, ci, ci, vp, cs, vp, vp, vp]
    L.qasr_encoder_host_pipeline_bytes.argtypes = [P(QasrLayer), ci, ci, ci, ci, P(cs)]
    L.qasr_encoder_host_pipeline_bytes.restype = ci
    L.qasr_encoder_forward_host_async.argtypes = [vp, P(QasrLayer), ci, vp, ci, ci, ci, vp, cs, vp, vp, vp, ci]
    L.qasr_encoder_forward_host_async.restype = ci
    L.qasr_encoder_host_wait.argtypes = [vp, ci]
    L.qasr_encoder_host_wait.restype = ci
    for name in ("qasr_create", "qasr_destroy", "qasr_poll_status", "qasr_set_option", "qasr_dw_conv", "qasr_conv",
                 "qasr_tcs_block_workspace_bytes", "qasr_tcs_block", "qasr_residual_requant_add",
                 "qasr_dequant_logits", "qasr_encoder_workspace_bytes", "qasr_encoder_forward",
                 "qasr_encoder_buffer_info", "qasr_encoder_host_staging_bytes", "qasr_encoder_forward_host"):
        getattr(L, name).restype = ci
    L.qasr_profile_read.argtypes = [vp, P(QasrProfileEntry), ci, P(ci)]
    L.qasr_profile_read.restype = ci
    L.qasr_kernel_name.argtypes = [ci]
    L.qasr_kernel_name.restype = ctypes.c_char_p
    L.qasr_layer_size.restype = ctypes.c_size_t
    L.qasr_layer_size.argtypes = []
    if L.qasr_layer_size() != ctypes.sizeof(QasrLayer):
        raise ImportError("qasr_layer layout mismatch between libqasr.so and the binding")
    _lib = L
    return L


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, torch.Tensor):
        assert t.is_contiguous(), "tensors must be contiguous"
        return t.data_ptr()
    return int(t)


def _rq(mult, shift):
    return QasrRequant(_ptr(mult), _ptr(shift))


def _terms(terms, mult, shift):
    n = len(terms)
    arr = (ctypes.c_void_p * max(n, 1))(*[_ptr(t) for t in terms])
    m = (ctypes.c_int32 * max(n, 1))(*[int(v) for v in mult])
    s = (ctypes.c_uint8 * max(n, 1))(*[int(v) for v in shift])
    return n, arr, m, s


NOALLOC_SCRATCH_BYTES = 16 << 20


def tcs_block_noalloc(x, w_dw, stride, dilation, m_dw, s_dw, w_pw, bias, max_abs_bias, m_pw, s_pw, relu, y,
                      device=0, stream=None, wait=True):
    """qasr_tcs_block_noalloc: the TCS block for callers that may not allocate device memory -- no
    context, no workspace; the depthwise output sits in the library's static device array (at most
    NOALLOC_SCRATCH_BYTES).  `y` must be supplied by the caller; nothing is allocated here either."""
    L = lib()
    B, C_in, T = x.shape
    if stream is None:
        stream = torch.cuda.current_stream(device).cuda_stream
    rc = L.qasr_tcs_block_noalloc(int(device), ctypes.c_void_p(stream), _ptr(x), B, C_in, T, _ptr(w_dw),
                                  w_dw.shape[1], stride, dilation, _rq(m_dw, s_dw), _ptr(w_pw), w_pw.shape[0],
                                  _ptr(bias), int(max_abs_bias), _rq(m_pw, s_pw), int(bool(relu)), _ptr(y),
                                  int(bool(wait)))
    if rc != 0:
        raise QasrError(rc, L.qasr_strerror(rc).decode())
    return y


class Context:
    """A qasr_ctx bound to one device and one stream (default: torch's current stream)."""

    def __init__(self, device=0, stream=None):
        self._lib = lib()
        self.device = int(device)
        if stream is None:
            stream = torch.cuda.current_stream(self.device).cuda_stream
        h = ctypes.c_void_p()
        rc = self._lib.qasr_create(ctypes.byref(h), self.device, ctypes.c_void_p(stream))
        if rc != 0:
            raise QasrError(rc, self._lib.qasr_strerror(rc).decode())
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._lib.qasr_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc):
        if rc != 0:
            raise QasrError(rc, self._lib.qasr_strerror(rc).decode(), self._lib.qasr_last_error(self._h).decode())

    # -- context calls
    def poll_status(self):
        self._check(self._lib.qasr_poll_status(self._h))

    def set_option(self, option, value):
        self._check(self._lib.qasr_set_option(self._h, int(option), int(value)))

    def selftest_wait_timeout(self, limit_us=1000):
        self._check(self._lib.qasr_selftest_wait_timeout(self._h, int(limit_us)))

    def measure_int8_tensor_peak(self, kblocks=20000):
        """Measured int8 tensor-core throughput in TOP/s (multiply-accumulate = 2 ops) and the device time in ms."""
        ms, ops = ctypes.c_float(), ctypes.c_double()
        self._check(self._lib.qasr_measure_int8_tensor_peak(self._h, int(kblocks), ctypes.byref(ms), ctypes.byref(ops)))
        return ops.value / (ms.value * 1e-3) / 1e12, ms.value

    def launch_count(self):
        return int(self._lib.qasr_launch_count(self._h))

    def profile_read(self, capacity=8192):
        """Records of the launches made in profile mode: list of dicts."""
        buf = (QasrProfileEntry * capacity)()
        n = ctypes.c_int()
        self._check(self._lib.qasr_profile_read(self._h, buf, capacity, ctypes.byref(n)))
        return [{"layer": e.layer, "kernel": self._lib.qasr_kernel_name(e.kernel).decode(), "ms": e.ms,
                 "macs": e.macs, "bytes": e.bytes} for e in buf[:min(n.value, capacity)]]

    # -- single operations (names follow include/qasr.h)
    def dw_conv(self, x, w_dw, stride, dilation, mult, shift, y=None):
        B, C, T = x.shape
        K = w_dw.shape[1]
        if y is None:
            y = torch.empty((B, C, (T - 1) // stride + 1), dtype=torch.int8, device=x.device)
        self._check(self._lib.qasr_dw_conv(self._h, _ptr(x), B, C, T, _ptr(w_dw), K, stride, dilation,
                                           _rq(mult, shift), _ptr(y)))
        return y

    def conv(self, x, w, bias, max_abs_bias, mult, shift, relu, stride=1, dilation=1,
             terms=(), term_mult=(), term_shift=(), out_int32=False, y=None):
        B, C_in, T = x.shape
        C_out = w.shape[0]
        K = w.shape[2] if w.dim() == 3 else 1
        T_out = (T - 1) // stride + 1
        if y is None:
            y = torch.empty((B, C_out, T_out), dtype=torch.int32 if out_int32 else torch.int8, device=x.device)
        n, arr, m, s = _terms(list(terms), term_mult, term_shift)
        self._check(self._lib.qasr_conv(self._h, _ptr(x), B, C_in, T, _ptr(w), C_out, K, stride, dilation,
                                        _ptr(bias), int(max_abs_bias), _rq(mult, shift), int(bool(relu)),
                                        n, arr, m, s,
                                        None if out_int32 else _ptr(y), _ptr(y) if out_int32 else None))
        return y

    def conv_scratch_bytes(self, B, C_in, C_out, T, K, stride=1):
        out = ctypes.c_size_t()
        self._check(self._lib.qasr_conv_scratch_bytes(B, C_in, C_out, T, K, stride, ctypes.byref(out)))
        return out.value

    def set_conv_scratch(self, scratch):
        """Lends a uint8 device tensor (or None) to later conv() calls; the context keeps it alive."""
        self._conv_scratch = scratch
        if scratch is None:
            self._check(self._lib.qasr_set_conv_scratch(self._h, None, 0))
        else:
            self._check(self._lib.qasr_set_conv_scratch(self._h, _ptr(scratch), scratch.numel()))

    def tcs_block_workspace_bytes(self, B, C_in, C_out, T, K, stride, dilation):
        out = ctypes.c_size_t()
        rc = self._lib.qasr_tcs_block_workspace_bytes(B, C_in, C_out, T, K, stride, dilation, ctypes.byref(out))
        self._check(rc)
        return out.value

    def tcs_block(self, x, w_dw, stride, dilation, m_dw, s_dw, w_pw, bias, max_abs_bias, m_pw, s_pw, relu,
                  y=None, workspace=None):
        B, C_in, T = x.shape
        K = w_dw.shape[1]
        C_out = w_pw.shape[0]
        if y is None:
            y = torch.empty((B, C_out, (T - 1) // stride + 1), dtype=torch.int8, device=x.device)
        if workspace is None:
            need = self.tcs_block_workspace_bytes(B, C_in, C_out, T, K, stride, dilation)
            workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=x.device)
        self._check(self._lib.qasr_tcs_block(self._h, _ptr(x), B, C_in, T, _ptr(w_dw), K, stride, dilation,
                                             _rq(m_dw, s_dw), _ptr(w_pw), C_out, _ptr(bias), int(max_abs_bias),
                                             _rq(m_pw, s_pw), int(bool(relu)), _ptr(y),
                                             _ptr(workspace), workspace.numel()))
        return y

    def residual_requant_add(self, terms, mult, shift, relu, y=None):
        B, C, T = terms[0].shape
        if y is None:
            y = torch.empty((B, C, T), dtype=torch.int8, device=terms[0].device)
        n, arr, m, s = _terms(list(terms), mult, shift)
        self._check(self._lib.qasr_residual_requant_add(self._h, n, arr, m, s, B, C, T, int(bool(relu)), _ptr(y)))
        return y

    def glu(self, x, q_c, mult, shift, y=None):
        B, C2, T = x.shape
        if y is None:
            y = torch.empty((B, C2 // 2, T), dtype=torch.int8, device=x.device)
        self._check(self._lib.qasr_glu(self._h, _ptr(x), B, C2 // 2, T, int(q_c), _rq(mult, shift), _ptr(y)))
        return y

    def dequant_logits(self, acc, scale, out=None):
        B, C, T = acc.shape
        if out is None:
            out = torch.empty((B, C, T), dtype=torch.float32, device=acc.device)
        self._check(self._lib.qasr_dequant_logits(self._h, _ptr(acc), B, C, T, _ptr(scale), _ptr(out)))
        return out

    # -- whole encoder
    def encoder_workspace_bytes(self, dm, B, T):
        out = ctypes.c_size_t()
        self._check(self._lib.qasr_encoder_workspace_bytes(dm.table, dm.n_layers, B, dm.C_in, T, ctypes.byref(out)))
        return out.value

    def encoder_host_staging_bytes(self, dm, B, T):
        out = ctypes.c_size_t()
        self._check(self._lib.qasr_encoder_host_staging_bytes(dm.table, dm.n_layers, B, dm.C_in, T, ctypes.byref(out)))
        return out.value

    def encoder_buffer_info(self, dm, B, T, buf_id):
        off, C, Tl = ctypes.c_size_t(), ctypes.c_int(), ctypes.c_int()
        self._check(self._lib.qasr_encoder_buffer_info(dm.table, dm.n_layers, B, dm.C_in, T, int(buf_id),
                                                       ctypes.byref(off), ctypes.byref(C), ctypes.byref(Tl)))
        return off.value, C.value, Tl.value

    def encoder_forward(self, dm, x, workspace, logits_q, logits=None):
        B, C_in, T = x.shape
        self._check(self._lib.qasr_encoder_forward(self._h, dm.table, dm.n_layers, _ptr(x), B, C_in, T,
                                                   _ptr(workspace), workspace.numel(), _ptr(logits_q),
                                                   _ptr(logits), _ptr(dm.out_scale) if logits is not None else None))
        return logits_q, logits

    def encoder_forward_host(self, dm, x_host, workspace, logits_q_host, logits_host=None):
        B, C_in, T = x_host.shape
        self._check(self._lib.qasr_encoder_forward_host(self._h, dm.table, dm.n_layers, _ptr(x_host), B, C_in, T,
                                                        _ptr(workspace), workspace.numel(), _ptr(logits_q_host),
                                                        _ptr(logits_host),
                                                        _ptr(dm.out_scale) if logits_host is not None else None))
        return logits_q_host, logits_host


    def encoder_host_pipeline_bytes(self, dm, B, T):
        out = ctypes.c_size_t()
        self._check(self._lib.qasr_encoder_host_pipeline_bytes(dm.table, dm.n_layers, B, dm.C_in, T, ctypes.byref(out)))
        return out.value

    def encoder_forward_host_async(self, dm, x_host, workspace, logits_q_host, logits_host=None, slot=0):
        B, C_in, T = x_host.shape
        self._check(self._lib.qasr_encoder_forward_host_async(self._h, dm.table, dm.n_layers, _ptr(x_host), B, C_in, T,
                                                              _ptr(workspace), workspace.numel(), _ptr(logits_q_host),
                                                              _ptr(logits_host),
                                                              _ptr(dm.out_scale) if logits_host is not None else None,
                                                              int(slot)))

    def encoder_host_wait(self, slot):
        self._check(self._lib.qasr_encoder_host_wait(self._h, int(slot)))


class DeviceModel:
    """A model description (see workloads/) with its constants uploaded to the device and its
    layer table laid out as an array of qasr_layer.  Marshalling only."""

    def __init__(self, model, device=0):
        self.device = torch.device("cuda", device) if not isinstance(device, torch.device) else device
        self.C_in = int(model["C_in"])
        self.layers = model["layers"]
        self.n_layers = len(self.layers)
        self._keep = []
        self.table = (QasrLayer * self.n_layers)()
        for i, L in enumerate(self.layers):
            e = self.table[i]
            e.kind = LAYER_KINDS[L["kind"]]
            e.in_buf = int(L.get("in", 0))
            e.out_buf = int(L["out"])
            e.C_in, e.C_out = int(L.get("C_in", 0)), int(L.get("C_out", 0))
            e.K, e.stride, e.dilation = int(L.get("K", 1)), int(L.get("stride", 1)), int(L.get("dilation", 1))
            if "w_dw" in L:
                e.w_dw = self._up(L["w_dw"], torch.int8)
                e.rq_dw = QasrRequant(self._up(L["m_dw"], torch.int32), self._up(L["s_dw"], torch.uint8))
            if "w" in L:
                e.w = self._up(L["w"], torch.int8)
                if L.get("bias") is not None:
                    e.bias = self._up(L["bias"], torch.int32)
                    e.max_abs_bias = int(L["max_abs_bias"])
                e.rq = QasrRequant(self._up(L["m"], torch.int32), self._up(L["s"], torch.uint8))
            if L["kind"] == "glu":
                e.glu_qc = int(L["q_c"])
                e.rq = QasrRequant(self._up(L["m"], torch.int32), self._up(L["s"], torch.uint8))
            e.relu = int(bool(L.get("relu", False)))
            e.out_int32 = int(bool(L.get("out_int32", False)))
            res = list(L.get("res") or [])
            if L["kind"] == "add":
                e.n_terms = len(res)
                for j, b in enumerate(res):
                    e.term_buf[j] = int(b)
            elif res:
                e.n_terms = 1 + len(res)
                for j, b in enumerate(res):
                    e.term_buf[j + 1] = int(b)
            for j in range(e.n_terms):
                e.term_mult[j] = int(L["res_m"][j])
                e.term_shift[j] = int(L["res_s"][j])
        self.out_scale = None
        if model.get("out_scale") is not None:
            self.out_scale = torch.from_numpy(np.ascontiguousarray(model["out_scale"], np.float32)).to(self.device)

    def _up(self, a, dtype):
        t = torch.from_numpy(np.ascontiguousarray(a)).to(dtype=dtype).contiguous().to(self.device)
        self._keep.append(t)
        return t.data_ptr()

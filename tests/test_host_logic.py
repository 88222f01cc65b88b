"""CPU-only checks of the product library: it builds, loads, exports every symbol the header
declares, and its host-side table validation / buffer planning behaves (no kernel is launched)."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def q():
    from paper_2103_16827_b200 import build as qbuild
    qbuild.build()
    import paper_2103_16827_b200 as pkg
    return pkg


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(qasr_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol(q):
    L = ctypes.CDLL(q.lib_path())
    names = _declared_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), "missing symbol " + n


def test_layer_struct_layout_matches(q):
    assert q.lib().qasr_layer_size() == ctypes.sizeof(q.QasrLayer)


def test_strerror_is_total(q):
    for code in range(-12, 1):
        assert q.lib().qasr_strerror(code)


def _table(q, layers):
    t = (q.QasrLayer * len(layers))()
    for i, d in enumerate(layers):
        for k, v in d.items():
            if k in ("term_buf", "term_mult", "term_shift"):
                for j, x in enumerate(v):
                    getattr(t[i], k)[j] = x
            elif k in ("rq", "rq_dw"):
                setattr(t[i], k, q.QasrRequant(*v))
            else:
                setattr(t[i], k, v)
    return t


def _ws(q, t, B, C_in, T):
    out = ctypes.c_size_t()
    rc = q.lib().qasr_encoder_workspace_bytes(t, len(t), B, C_in, T, ctypes.byref(out))
    return rc, out.value


FAKE = 0x1000  # never dereferenced by the planning code


def _pw(i, o, ci, co, **kw):
    d = dict(kind=2, in_buf=i, out_buf=o, C_in=ci, C_out=co, K=1, stride=1, dilation=1, w=FAKE, bias=FAKE,
             max_abs_bias=4096, rq=(FAKE, FAKE), relu=1)
    d.update(kw)
    return d


def _tcs(i, o, ci, co, K, stride=1, dilation=1, **kw):
    d = dict(kind=4, in_buf=i, out_buf=o, C_in=ci, C_out=co, K=K, stride=stride, dilation=dilation, w_dw=FAKE,
             rq_dw=(FAKE, FAKE), w=FAKE, bias=FAKE, max_abs_bias=4096, rq=(FAKE, FAKE), relu=1)
    d.update(kw)
    return d


def test_workspace_planning_sizes_and_buffer_info(q):
    B, T = 3, 100
    layers = [_tcs(0, 1, 64, 256, 33, stride=2), _pw(1, 2, 256, 512), _tcs(2, 1, 512, 512, 87, dilation=2),
              _pw(1, 3, 512, 29, out_int32=1, relu=0)]
    t = _table(q, layers)
    rc, total = _ws(q, t, B, 64, T)
    assert rc == 0
    up = lambda v: (v + 255) // 256 * 256
    b1 = max(B * 256 * 50, B * 512 * 50)       # buffer 1 is written twice
    b2 = B * 512 * 50
    # scratch: depthwise outputs of the two TCS layers, frame-major input copies of the two stand-alone
    # convolutions (T = 50 is not a multiple of 16, so they take the implicit-GEMM path); behind it one region
    # per such layer for its regrouped weights
    scratch = max(B * 64 * 50, B * 512 * 50, up(B * 256 * 50), up(B * 512 * 50))
    # a second region as large as the largest frame-major input copy of a stride-1 layer: a convolution's epilogue
    # writes the next one's copy there while it reads its own from the first
    scratch2 = max(up(B * 256 * 50), up(B * 512 * 50))
    assert total == up(b1) + up(b2) + up(scratch) + up(scratch2) + up(512 * 256) + up(29 * 512)
    off, C, Tl = ctypes.c_size_t(), ctypes.c_int(), ctypes.c_int()
    rc = q.lib().qasr_encoder_buffer_info(t, len(t), B, 64, T, 2, ctypes.byref(off), ctypes.byref(C), ctypes.byref(Tl))
    assert rc == 0 and off.value == up(b1) and C.value == 512 and Tl.value == 50


@pytest.mark.parametrize("mutate,code", [
    (lambda L: L[1].update(in_buf=7), -9),                  # reads a buffer nobody wrote
    (lambda L: L[1].update(C_in=128), -9),                  # channel mismatch
    (lambda L: L[1].update(out_buf=1), -9),                 # in place
    (lambda L: L[0].update(K=32), -2),                      # even kernel
    (lambda L: L[0].update(stride=3), -2),
    (lambda L: L[0].update(out_int32=1), -9),               # int32 output before the end
    (lambda L: L[2].update(out_int32=0), -9),               # last layer must give logits
    (lambda L: L[1].update(w=0), -1),
    (lambda L: L[1].update(max_abs_bias=2 ** 31 - 1), -5),  # overflow cannot be excluded
    (lambda L: L[1].update(n_terms=2, term_buf=[0, 9], term_mult=[1, 1], term_shift=[1, 1]), -9),
    (lambda L: L[1].update(n_terms=2, term_buf=[0, 1], term_mult=[1, 1], term_shift=[1, 1]), -9),  # wrong shape
    (lambda L: L[1].update(kind=9), -9),
])
def test_table_validation_rejects_bad_tables(q, mutate, code):
    layers = [_tcs(0, 1, 64, 256, 33, stride=2), _pw(1, 2, 256, 512), _pw(2, 3, 512, 29, out_int32=1, relu=0)]
    mutate(layers)
    rc, _ = _ws(q, _table(q, layers), 2, 64, 64)
    assert rc == code


def test_residual_term_range_is_checked_on_the_host(q):
    layers = [_pw(0, 1, 64, 64), _pw(1, 2, 64, 64, n_terms=2, term_buf=[0, 1], term_mult=[1, 1], term_shift=[1, 63]),
              _pw(2, 3, 64, 29, out_int32=1, relu=0)]
    rc, _ = _ws(q, _table(q, layers), 2, 64, 64)
    assert rc == -4


def test_device_model_marshals_the_quartznet_table(q):
    import workloads
    model, x = workloads.quartznet_model(2, 64, repeat=1, variant="live", seed=3)
    # build the table without touching a GPU: same marshalling, fake pointers
    names = [L["name"] for L in model["layers"]]
    assert names[0] == "C1" and names[-1] == "C4" and len(names) == 1 + 5 * 6 + 3
    assert model["n_bufs"] <= 5
    last = model["layers"][-1]
    assert last["out_int32"] and not last["relu"]
    res_layers = [L for L in model["layers"] if L["res"]]
    assert len(res_layers) == 5 and all(L["name"].endswith(".4") for L in res_layers)


def test_tcs_block_workspace_bytes(q):
    out = ctypes.c_size_t()
    assert q.lib().qasr_tcs_block_workspace_bytes(2, 64, 256, 101, 33, 2, 1, ctypes.byref(out)) == 0
    assert out.value == (2 * 64 * 51 + 255) // 256 * 256
    assert q.lib().qasr_tcs_block_workspace_bytes(2, 64, 256, 101, 32, 2, 1, ctypes.byref(out)) == -2


def test_conv_scratch_bytes_counts_the_frame_major_copy_and_the_regrouped_weights(q):
    out = ctypes.c_size_t()
    up = lambda v: (v + 255) // 256 * 256
    # stride 1: one plane of T rows; stride 2: two planes of ceil(T / 2) rows
    assert q.lib().qasr_conv_scratch_bytes(3, 48, 40, 100, 11, 1, ctypes.byref(out)) == 0
    assert out.value == up(3 * 100 * 48) + up(11 * 40 * 48)
    assert q.lib().qasr_conv_scratch_bytes(2, 16, 8, 101, 5, 2, ctypes.byref(out)) == 0
    assert out.value == up(2 * 2 * 51 * 16) + up(5 * 8 * 16)
    # errors are codes: NULL result, even K, bad stride, non-positive sizes
    assert q.lib().qasr_conv_scratch_bytes(1, 16, 16, 16, 3, 1, None) == -1
    assert q.lib().qasr_conv_scratch_bytes(1, 16, 16, 16, 4, 1, ctypes.byref(out)) == -2
    assert q.lib().qasr_conv_scratch_bytes(1, 16, 16, 16, 3, 3, ctypes.byref(out)) == -2
    assert q.lib().qasr_conv_scratch_bytes(0, 16, 16, 16, 3, 1, ctypes.byref(out)) == -2
    assert q.lib().qasr_set_conv_scratch(None, None, 0) == -1

"""Seeded synthetic inputs and model descriptions for the Q-ASR integer-only path.

This module only DRAWS inputs: int8 activations, int8 weights, int32 biases,
dyadic multipliers/shifts and the layer tables of the encoder shapes.  It holds
none of the inference arithmetic (no convolution, no requantisation) and is the
only module shared by the CPU oracle's tests and the GPU library's tests.

The trained models and the speech corpus the paper evaluates on are not
available, so every tensor is synthetic: shapes follow the QuartzNet / Jasper /
Conformer encoders the paper quantises (Sec. 3), value distributions follow the
single-block configuration (int8 input quantised from N(0,1) with scale 0.05,
weights uniform in [-127,127], bias uniform in [-2^12, 2^12], multipliers
uniform in [2^14, 2^15)).

Two scale variants:
  literal  shift = 30 everywhere.  With these numbers every activation rounds to
           zero after one or two layers, so this variant only proves that the
           degenerate case is handled.
  live     the same multiplier draws, but each channel's shift is chosen from the
           expected accumulator spread (closed form from the input/weight second
           moments) so that outputs span the int8 range with a little
           saturation, the way a min/max-calibrated model (Sec. 3.1) would.

A model description is a dict {"name", "B", "T", "C_in", "layers": [...],
"out_scale": float32[C_last], "n_bufs"}; each layer is a dict with
  kind    "tcs" | "dw" | "pw" | "dense" | "add" | "glu" (q_c, m, s: the integer gate of the Conformer module)
  in/out  activation buffer ids (0 is the encoder input)
  C_in, C_out, K, stride, dilation
  w_dw int8[C_in][K], m_dw int32[C_in], s_dw uint8[C_in]           (tcs, dw)
  w int8[C_out][C_in] or [C_out][C_in][K], bias int32[C_out], max_abs_bias,
  m int32[C_out], s uint8[C_out]                                    (tcs, pw, dense)
  relu, out_int32
  res [buffer ids], res_m int32[1+len(res)], res_s uint8[1+len(res)]  (index 0 = main branch)
Draw order (fixed): encoder input first, then for each layer in table order
w_dw, m_dw, w, bias, m, residual multipliers; out_scale last.
"""
from __future__ import annotations

import math

import numpy as np

W_MS = (255.0 ** 2 - 1.0) / 12.0      # second moment of an integer uniform on [-127, 127]
TARGET = 44.0                          # aimed-at std (in int8 steps) of a pre-activation, live variant
G2 = 1.0404                            # E[g^2] of the per-channel gain spread g in [1/sqrt2, sqrt2)
MS_LIN = TARGET * TARGET * G2          # second moment of a requantised tensor without ReLU
MS_RELU = MS_LIN / 2.0                 # ... after ReLU (zero-mean symmetric pre-activation)
MS_INPUT = 400.0                       # N(0,1) / 0.05
MAX_RES = 12


def rng_for(seed: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(seed))


def draw_input(rng, B, C, T):
    """int8 activations quantised from N(0,1) with scale 0.05 (round half away, clamp)."""
    x = rng.standard_normal((B, C, T), dtype=np.float32).astype(np.float64) / 0.05
    q = np.sign(x) * np.floor(np.abs(x) + 0.5)
    return np.clip(q, -128, 127).astype(np.int8)


def draw_weights(rng, shape):
    return rng.integers(-127, 128, size=shape, dtype=np.int64).astype(np.int8)


def draw_bias(rng, C):
    return rng.integers(-(1 << 12), (1 << 12) + 1, size=C, dtype=np.int64).astype(np.int32)


def _live_shift(mult, acc_rms, target):
    """Shift s so that mult / 2^s * acc_rms lands within a factor sqrt(2) of target."""
    s = np.rint(np.log2(mult.astype(np.float64) * acc_rms / target)).astype(np.int64)
    return np.clip(s, 1, 62).astype(np.uint8)


def draw_requant(rng, C, variant, acc_rms):
    mult = rng.integers(1 << 14, 1 << 15, size=C, dtype=np.int64).astype(np.int32)
    if variant == "literal":
        shift = np.full(C, 30, dtype=np.uint8)
    elif variant == "live":
        shift = _live_shift(mult, acc_rms, TARGET)
    else:
        raise ValueError(variant)
    return mult, shift


def draw_residual_scales(rng, n_terms, variant):
    """Per-term (per-tensor) dyadic numbers for the integer residual add."""
    if variant == "literal":
        mult = rng.integers(1 << 14, 1 << 15, size=n_terms, dtype=np.int64).astype(np.int32)
        shift = np.full(n_terms, 30, dtype=np.uint8)
        return mult, shift
    u = rng.uniform(0.9, 1.1, size=n_terms) / math.sqrt(n_terms)
    mult = np.empty(n_terms, dtype=np.int32)
    shift = np.empty(n_terms, dtype=np.uint8)
    for j, M in enumerate(u):
        s = 0
        while M * (1 << s) < (1 << 14):
            s += 1
        m = int(math.floor(M * (1 << s) + 0.5))
        if m >= (1 << 15):
            m >>= 1
            s -= 1
        mult[j], shift[j] = m, s
    return mult, shift


class _Builder:
    """Accumulates layers, handing out buffer ids (ping-pong, or one per layer)."""

    def __init__(self, rng, variant, unique_bufs, split_tcs):
        self.rng = rng
        self.variant = variant
        self.unique = unique_bufs
        self.split = split_tcs
        self.layers = []
        self.next_buf = 1
        self.free = []

    def new_buf(self):
        if not self.unique and self.free:
            return self.free.pop()
        b = self.next_buf
        self.next_buf += 1
        return b

    def release(self, b):
        if not self.unique and b != 0 and b not in self.free:
            self.free.append(b)

    # -- layer makers; ms_in is the expected second moment of the input tensor
    def conv(self, kind, name, src, C_in, C_out, K, stride, dilation, relu, ms_in,
             res=None, out_int32=False):
        rng, v = self.rng, self.variant
        L = {"name": name, "kind": kind, "in": src, "C_in": C_in, "C_out": C_out, "K": K,
             "stride": stride, "dilation": dilation, "relu": bool(relu), "out_int32": bool(out_int32),
             "res": list(res or [])}
        if kind in ("tcs", "dw"):
            L["w_dw"] = draw_weights(rng, (C_in, K))
            L["m_dw"], L["s_dw"] = draw_requant(rng, C_in, v, math.sqrt(K * W_MS * ms_in))
            ms_mid = MS_LIN
            taps = C_in
        else:
            ms_mid = ms_in
            taps = C_in * K
        if kind != "dw":
            wshape = (C_out, C_in) if kind in ("tcs", "pw") else (C_out, C_in, K)
            L["w"] = draw_weights(rng, wshape)
            L["bias"] = draw_bias(rng, C_out)
            L["max_abs_bias"] = int(np.abs(L["bias"].astype(np.int64)).max())
            L["m"], L["s"] = draw_requant(rng, C_out, v, math.sqrt(taps * W_MS * ms_mid))
        if L["res"]:
            assert len(L["res"]) + 1 <= MAX_RES
            L["res_m"], L["res_s"] = draw_residual_scales(rng, 1 + len(L["res"]), v)
        L["out"] = self.new_buf()
        self.layers.append(L)
        return L["out"]

    def tcs(self, name, src, C_in, C_out, K, stride, dilation, relu, ms_in, res=None):
        if not self.split:
            return self.conv("tcs", name, src, C_in, C_out, K, stride, dilation, relu, ms_in, res)
        # the same draws, emitted as a depthwise layer followed by a pointwise layer
        rng, v = self.rng, self.variant
        d = {"name": name + ".dw", "kind": "dw", "in": src, "C_in": C_in, "C_out": C_in, "K": K,
             "stride": stride, "dilation": dilation, "relu": False, "out_int32": False, "res": []}
        d["w_dw"] = draw_weights(rng, (C_in, K))
        d["m_dw"], d["s_dw"] = draw_requant(rng, C_in, v, math.sqrt(K * W_MS * ms_in))
        d["out"] = self.new_buf()
        self.layers.append(d)
        p = {"name": name + ".pw", "kind": "pw", "in": d["out"], "C_in": C_in, "C_out": C_out, "K": 1,
             "stride": 1, "dilation": 1, "relu": bool(relu), "out_int32": False, "res": list(res or [])}
        p["w"] = draw_weights(rng, (C_out, C_in))
        p["bias"] = draw_bias(rng, C_out)
        p["max_abs_bias"] = int(np.abs(p["bias"].astype(np.int64)).max())
        p["m"], p["s"] = draw_requant(rng, C_out, v, math.sqrt(C_in * W_MS * MS_LIN))
        if p["res"]:
            p["res_m"], p["res_s"] = draw_residual_scales(rng, 1 + len(p["res"]), v)
        p["out"] = self.new_buf()
        self.layers.append(p)
        self.release(d["out"])
        return p["out"]


def tcs_block_model(B=1, T=256, C=256, K=33, variant="live", seed=0):
    """One QuartzNet time-channel-separable block on an int8 input [B][C][T]:
    depthwise K taps, pointwise 1x1 with folded-BN bias, requant, ReLU."""
    rng = rng_for(seed)
    x = draw_input(rng, B, C, T)
    bld = _Builder(rng, variant, True, False)
    bld.conv("tcs", "block", 0, C, C, K, 1, 1, True, MS_INPUT)
    return {"name": "tcs_block", "B": B, "T": T, "C_in": C, "layers": bld.layers,
            "out_scale": None, "n_bufs": bld.next_buf, "variant": variant}, x


QUARTZ_CHANNELS = (256, 256, 512, 512, 512)
QUARTZ_KERNELS = (33, 39, 51, 63, 75)


def quartznet_model(B, T, repeat=1, variant="live", seed=1, mel=64, unique_bufs=False,
                    split_tcs=False, channels=QUARTZ_CHANNELS, kernels=QUARTZ_KERNELS,
                    c1=256, c2=512, c3=1024, n_out=29, subblocks=5):
    """QuartzNet-(5*repeat)x5-shaped encoder.

    C1 (TCS, K=33, stride 2) -> for each of the 5 block shapes, `repeat` blocks of
    `subblocks` TCS sub-blocks; every block adds a 1x1-conv projection of its own
    input to the last sub-block's output before the last ReLU -> C2 (TCS, K=87,
    dilation 2) -> C3 (1x1, c3) -> C4 (1x1, n_out, int32 logits, no ReLU).
    """
    rng = rng_for(seed)
    x = draw_input(rng, B, mel, T)
    bld = _Builder(rng, variant, unique_bufs, split_tcs)
    cur = bld.tcs("C1", 0, mel, c1, 33, 2, 1, True, MS_INPUT)
    cin = c1
    for bi, (c, k) in enumerate(zip(channels, kernels)):
        for r in range(repeat):
            tag = "B%d.%d" % (bi, r)
            # residual branch first, while the block input is the freshest tensor
            rbuf = bld.conv("pw", tag + ".res", cur, cin, c, 1, 1, 1, False, MS_RELU)
            h = cur
            for s in range(subblocks):
                last = s == subblocks - 1
                nxt = bld.tcs("%s.%d" % (tag, s), h, cin if s == 0 else c, c, k, 1, 1, True, MS_RELU,
                              res=[rbuf] if last else None)
                if h != cur:
                    bld.release(h)
                h = nxt
            # the block input keeps its buffer until the block ends: the projection that reads it may then run
            # beside the sub-blocks instead of in front of them (nothing overwrites its input meanwhile)
            bld.release(cur)
            bld.release(rbuf)
            cur = h
            cin = c
    nxt = bld.tcs("C2", cur, cin, c2, 87, 1, 2, True, MS_RELU)
    bld.release(cur)
    cur = nxt
    nxt = bld.conv("pw", "C3", cur, c2, c3, 1, 1, 1, True, MS_RELU)
    bld.release(cur)
    cur = nxt
    bld.conv("pw", "C4", cur, c3, n_out, 1, 1, 1, False, MS_RELU, out_int32=True)
    out_scale = (rng.uniform(0.5, 1.5, size=n_out) * 1e-3).astype(np.float32)
    name = "quartznet%dx%d" % (len(channels) * repeat, subblocks)
    return {"name": name, "B": B, "T": T, "C_in": mel, "layers": bld.layers, "out_scale": out_scale,
            "n_bufs": bld.next_buf, "variant": variant}, x


JASPER_CHANNELS = (256, 256, 384, 384, 512, 512, 640, 640, 768, 768)
JASPER_KERNELS = (11, 11, 13, 13, 17, 17, 21, 21, 25, 25)


def jasper_model(B, T, variant="live", seed=3, mel=64, unique_bufs=False, channels=JASPER_CHANNELS,
                 kernels=JASPER_KERNELS, c1=256, k1=11, c2=896, k2=29, c3=1024, n_out=29, subblocks=5):
    """JasperDR-(len(channels))x(subblocks)-shaped encoder with dense residuals.

    C1 (dense conv, K=k1, stride 2) -> blocks of `subblocks` dense K-tap conv sub-blocks; the last
    sub-block of block i adds, before its ReLU, a 1x1-conv projection of C1's output and of every
    earlier block's output (each rescaled by its own dyadic number) -> C2 (dense, K=k2,
    dilation 2) -> C3 (1x1) -> C4 (1x1, int32 logits).
    """
    rng = rng_for(seed)
    x = draw_input(rng, B, mel, T)
    bld = _Builder(rng, variant, unique_bufs, False)
    cur = bld.conv("dense", "C1", 0, mel, c1, k1, 2, 1, True, MS_INPUT)
    outs = [(cur, c1)]                       # tensors every later block draws a residual from
    cin = c1
    for bi, (c, k) in enumerate(zip(channels, kernels)):
        tag = "B%d" % bi
        rbufs = [bld.conv("pw", "%s.res%d" % (tag, j), src, sc, c, 1, 1, 1, False, MS_RELU)
                 for j, (src, sc) in enumerate(outs)]
        h = cur
        for s in range(subblocks):
            last = s == subblocks - 1
            nxt = bld.conv("dense", "%s.%d" % (tag, s), h, cin if s == 0 else c, c, k, 1, 1, True, MS_RELU,
                           res=rbufs if last else None)
            if h != cur:
                bld.release(h)               # block outputs stay alive: later blocks read them
            h = nxt
        for r in rbufs:
            bld.release(r)
        cur = h
        cin = c
        outs.append((cur, c))
    cur = bld.conv("dense", "C2", cur, cin, c2, k2, 1, 2, True, MS_RELU)
    cur = bld.conv("pw", "C3", cur, c2, c3, 1, 1, 1, True, MS_RELU)
    bld.conv("pw", "C4", cur, c3, n_out, 1, 1, 1, False, MS_RELU, out_int32=True)
    out_scale = (rng.uniform(0.5, 1.5, size=n_out) * 1e-3).astype(np.float32)
    return {"name": "jasper%dx%d" % (len(channels), subblocks), "B": B, "T": T, "C_in": mel, "layers": bld.layers,
            "out_scale": out_scale, "n_bufs": bld.next_buf, "variant": variant}, x


GLU_QC = 117           # gate saturates at |g| = 117 int8 steps (4 / 0.034)
GLU_SIG_MS = 0.33      # E[sigmoid^2] of a zero-mean gate with that spread


def conformer_model(B, T, variant="live", seed=4, d=256, layers=16, K=31, ff=4, n_out=29, unique_bufs=False):
    """Conformer-shaped convolution module + feed-forward stack on an int8 input [B][d][T]
    (already subsampled): per layer  pointwise d -> 2d, integer GLU -> d, TCS (depthwise K taps with the
    BatchNorm folded, pointwise d -> d) added to the layer input, pointwise d -> ff*d with ReLU,
    pointwise ff*d -> d added to its input; a final 1x1 head leaves int32 logits."""
    rng = rng_for(seed)
    x = draw_input(rng, B, d, T)
    bld = _Builder(rng, variant, unique_bufs, False)
    cur, ms_cur = 0, MS_INPUT
    for li in range(layers):
        tag = "L%d" % li
        e = bld.conv("pw", tag + ".pw1", cur, d, 2 * d, 1, 1, 1, False, ms_cur)
        g = {"name": tag + ".glu", "kind": "glu", "in": e, "C_in": 2 * d, "C_out": d, "K": 1, "stride": 1,
             "dilation": 1, "relu": False, "out_int32": False, "res": [], "q_c": GLU_QC}
        g["m"], g["s"] = draw_requant(rng, d, variant, math.sqrt(MS_LIN * GLU_SIG_MS) * 2 * GLU_QC * GLU_QC)
        g["out"] = bld.new_buf()
        bld.layers.append(g)
        bld.release(e)
        c = bld.tcs(tag + ".conv", g["out"], d, d, K, 1, 1, False, MS_LIN, res=[cur])
        bld.release(g["out"])
        if cur != 0:
            bld.release(cur)
        f1 = bld.conv("pw", tag + ".ff1", c, d, ff * d, 1, 1, 1, True, MS_LIN)
        f2 = bld.conv("pw", tag + ".ff2", f1, ff * d, d, 1, 1, 1, False, MS_RELU, res=[c])
        bld.release(f1)
        bld.release(c)
        cur, ms_cur = f2, MS_LIN
    bld.conv("pw", "head", cur, d, n_out, 1, 1, 1, False, MS_LIN, out_int32=True)
    out_scale = (rng.uniform(0.5, 1.5, size=n_out) * 1e-3).astype(np.float32)
    return {"name": "conformer_conv_ffn_x%d" % layers, "B": B, "T": T, "C_in": d, "layers": bld.layers,
            "out_scale": out_scale, "n_bufs": bld.next_buf, "variant": variant}, x


# The benchmark configurations, by index
def config(idx, variant="live", **kw):
    if idx == 0:
        return tcs_block_model(1, 256, 256, 33, variant=variant, seed=0)
    if idx == 1:
        return quartznet_model(kw.pop("B", 8), kw.pop("T", 1024), 1, variant=variant, seed=1, **kw)
    if idx == 2:
        return quartznet_model(kw.pop("B", 32), kw.pop("T", 1600), 3, variant=variant, seed=2, **kw)
    if idx == 3:
        return jasper_model(kw.pop("B", 16), kw.pop("T", 1600), variant=variant, seed=3, **kw)
    if idx == 4:
        return conformer_model(kw.pop("B", 16), kw.pop("T", 800), variant=variant, seed=4, **kw)
    raise ValueError("unknown config %r" % (idx,))


def model_stats(model):
    """MACs and int8 weight bytes of a model description (for the size/BOPs cross-check)."""
    T = model["T"]
    t_of = {0: T}
    macs = 0
    weights = 0
    for L in model["layers"]:
        if L["kind"] == "add":
            t_of[L["out"]] = t_of[L["res"][0]]
            continue
        if L["kind"] == "glu":
            t_of[L["out"]] = t_of[L["in"]]
            continue
        t_in = t_of[L["in"]]
        t_out = (t_in - 1) // L["stride"] + 1
        t_of[L["out"]] = t_out
        if L["kind"] in ("tcs", "dw"):
            macs += L["C_in"] * L["K"] * t_out
            weights += L["C_in"] * L["K"]
        if L["kind"] in ("tcs", "pw"):
            macs += L["C_in"] * L["C_out"] * t_out
            weights += L["C_in"] * L["C_out"]
        if L["kind"] == "dense":
            macs += L["C_in"] * L["C_out"] * L["K"] * t_out
            weights += L["C_in"] * L["C_out"] * L["K"]
    return {"macs_per_utterance": macs, "weights": weights, "T_out": t_out}

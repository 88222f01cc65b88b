"""Pins for the CPU oracle: each test checks it against something other than itself --
exact rational arithmetic, float64 library convolution (exact at these magnitudes),
closed forms, special cases and invariants -- chosen so that a dropped term, a wrong
sign or index, or a transposed operand fails at least one of them."""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle
import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ rounding shift RS
def _rs_exact(v, c):
    """round-half-up of the exact rational v / 2^c"""
    return math.floor(Fraction(v, 1 << c) + Fraction(1, 2))


def test_rs_matches_exact_rational_rounding():
    rng = np.random.default_rng(11)
    for _ in range(4000):
        c = int(rng.integers(1, 63))
        mag = int(rng.integers(1, 62))
        v = int(rng.integers(-(1 << mag), (1 << mag) + 1))
        assert oracle.rs(v, c) == _rs_exact(v, c), (v, c)


def test_rs_ties_go_up_and_exact_multiples():
    for c in (1, 2, 7, 30, 31, 32, 33, 62):
        half = 1 << (c - 1)
        assert oracle.rs(half, c) == 1
        assert oracle.rs(-half, c) == 0
        assert oracle.rs(half - 1, c) == (0 if c > 1 else 0)
        assert oracle.rs(-half - 1, c) == -1
        assert oracle.rs(0, c) == 0
        for k in (-5, -1, 1, 3):
            if abs(k) << c < (1 << 62):
                assert oracle.rs(k << c, c) == k
    # 3/2 -> 2, -3/2 -> -1, 5/2 -> 3, -5/2 -> -2 (half-up, not half-away, not half-even)
    assert [oracle.rs(v, 1) for v in (3, -3, 5, -5)] == [2, -1, 3, -2]


def test_rs_error_at_most_half_and_monotone():
    rng = np.random.default_rng(12)
    for _ in range(200):
        c = int(rng.integers(1, 40))
        base = int(rng.integers(-(1 << 45), 1 << 45))
        prev = None
        for v in range(base, base + 64):
            r = oracle.rs(v, c)
            assert abs(Fraction(r) - Fraction(v, 1 << c)) <= Fraction(1, 2)
            if prev is not None:
                assert r >= prev
            prev = r


def test_requant_within_one_lsb_of_float_rescaling_exhaustive_range():
    """mult = round(M * 2^c) with mult >= 2^14: the integer result stays within 1 LSB of a*M."""
    rng = np.random.default_rng(13)
    a = np.arange(-(1 << 17), (1 << 17) + 1, dtype=np.int32).reshape(1, 1, -1)
    for _ in range(64):
        M = float(2.0 ** rng.uniform(-16, -6))
        mult, shift = oracle.dyadic_encode(M)
        assert (1 << 14) <= mult < (1 << 15)
        y = oracle.requant(a, np.array([mult], np.int32), np.array([shift], np.uint8)).astype(np.float64)
        ref = np.clip(a.astype(np.float64) * M, -128, 127)
        inr = (np.abs(a.astype(np.float64) * M) < 126)
        assert np.max(np.abs(y - ref)[inr]) <= 0.5 + 128 * 2.0 ** -15 + 1e-9
        assert np.max(np.abs(y - ref)) < 1.0
        # and exactly equal to the rational definition on a sample
        for i in rng.integers(0, a.size, 50):
            v = int(a[0, 0, i])
            want = max(-128, min(127, _rs_exact(v * mult, shift)))
            assert int(y[0, 0, i]) == want


def test_requant_large_accumulators_and_wide_multipliers():
    rng = np.random.default_rng(14)
    acc = rng.integers(-(1 << 31), 1 << 31, size=(2, 3, 40), dtype=np.int64).astype(np.int32)
    mult = np.array([(1 << 31) - 1, 1, 12345], np.int32)
    shift = np.array([62, 1, 33], np.uint8)
    y = oracle.requant(acc, mult, shift)
    for b in range(2):
        for c in range(3):
            for t in range(40):
                want = max(-128, min(127, _rs_exact(int(acc[b, c, t]) * int(mult[c]), int(shift[c]))))
                assert int(y[b, c, t]) == want


def test_saturation_boundaries_and_relu():
    acc = np.array([126, 127, 128, 129, -127, -128, -129, -130, 0, -1, 1, 2 ** 31 - 1, -2 ** 31],
                   dtype=np.int64).astype(np.int32).reshape(1, 1, -1)
    one = np.array([1 << 20], np.int32)
    sh = np.array([20], np.uint8)
    y = oracle.requant(acc, one, sh)[0, 0]
    assert y.tolist() == [126, 127, 127, 127, -127, -128, -128, -128, 0, -1, 1, 127, -128]
    yr = oracle.requant(acc, one, sh, relu=True)[0, 0]
    assert yr.tolist() == [126, 127, 127, 127, 0, 0, 0, 0, 0, 0, 1, 127, 0]
    assert oracle.sat8(127) == 127 and oracle.sat8(128) == 127
    assert oracle.sat8(-128) == -128 and oracle.sat8(-129) == -128


# ------------------------------------------------------------------ integer convolution
def _torch_conv(x, w, bias, stride, dilation, depthwise):
    xt = torch.from_numpy(x.astype(np.float64))
    wt = torch.from_numpy(w.astype(np.float64))
    K = w.shape[-1]
    if depthwise:
        wt = wt.reshape(w.shape[0], 1, K)
        groups = w.shape[0]
    else:
        groups = 1
    bt = None if bias is None else torch.from_numpy(bias.astype(np.float64))
    y = torch.nn.functional.conv1d(xt, wt, bt, stride=stride, padding=dilation * (K - 1) // 2,
                                   dilation=dilation, groups=groups)
    return y.numpy()


@pytest.mark.parametrize("B,Ci,Co,T,K,stride,dil,dw", [
    (2, 5, 7, 37, 1, 1, 1, False),
    (2, 5, 7, 37, 3, 1, 1, False),
    (1, 3, 4, 50, 33, 1, 1, False),
    (2, 4, 6, 41, 5, 2, 1, False),
    (2, 4, 6, 40, 5, 2, 2, False),
    (3, 6, 6, 64, 33, 1, 1, True),
    (2, 6, 6, 63, 33, 2, 1, True),
    (2, 5, 5, 70, 9, 1, 2, True),
    (1, 5, 5, 9, 33, 1, 1, True),      # kernel wider than the signal
    (1, 2, 2, 1, 3, 1, 1, True),       # single frame
])
def test_conv_matches_float64_library_convolution(B, Ci, Co, T, K, stride, dil, dw):
    rng = np.random.default_rng(100 + K + T)
    x = rng.integers(-128, 128, size=(B, Ci, T)).astype(np.int8)
    w = rng.integers(-127, 128, size=(Co, K) if dw else (Co, Ci, K)).astype(np.int8)
    bias = rng.integers(-4096, 4097, size=Co).astype(np.int32)
    for b in (None, bias):
        acc = oracle.conv1d(x, w, b, stride, dil, depthwise=dw)
        ref = _torch_conv(x, w, b, stride, dil, dw)
        assert acc.shape == ref.shape == (B, Co, (T - 1) // stride + 1)
        assert np.array_equal(acc.astype(np.float64), ref)


def test_conv_brute_force_tiny():
    rng = np.random.default_rng(5)
    B, Ci, Co, T, K, stride, dil = 1, 2, 3, 11, 5, 2, 2
    x = rng.integers(-128, 128, size=(B, Ci, T)).astype(np.int8)
    w = rng.integers(-127, 128, size=(Co, Ci, K)).astype(np.int8)
    acc = oracle.conv1d(x, w, None, stride, dil)
    pad = dil * (K - 1) // 2
    for o in range(Co):
        for t in range((T - 1) // stride + 1):
            s = 0
            for i in range(Ci):
                for k in range(K):
                    ti = t * stride + k * dil - pad
                    if 0 <= ti < T:
                        s += int(w[o, i, k]) * int(x[0, i, ti])
            assert int(acc[0, o, t]) == s


def test_delta_kernel_is_a_shifted_copy():
    rng = np.random.default_rng(6)
    x = rng.integers(-128, 128, size=(2, 3, 20)).astype(np.int8)
    K = 7
    for k0 in range(K):
        w = np.zeros((3, K), np.int8)
        w[:, k0] = 1
        acc = oracle.conv1d(x, w, None, 1, 1, depthwise=True)
        off = k0 - (K - 1) // 2
        ref = np.zeros_like(acc)
        for t in range(20):
            if 0 <= t + off < 20:
                ref[:, :, t] = x[:, :, t + off]
        assert np.array_equal(acc, ref)


def test_identity_pointwise_with_unit_multiplier_returns_input():
    rng = np.random.default_rng(7)
    C = 6
    x = rng.integers(-128, 128, size=(2, C, 15)).astype(np.int8)
    w = np.eye(C, dtype=np.int8)
    acc = oracle.conv1d(x, w, None)
    y = oracle.requant(acc, np.full(C, 1 << 16, np.int32), np.full(C, 16, np.uint8))
    assert np.array_equal(y, x)


def test_accumulator_is_linear_in_the_input():
    rng = np.random.default_rng(8)
    x1 = rng.integers(-60, 60, size=(1, 4, 30)).astype(np.int8)
    x2 = rng.integers(-60, 60, size=(1, 4, 30)).astype(np.int8)
    w = rng.integers(-127, 128, size=(5, 4, 3)).astype(np.int8)
    a12 = oracle.conv1d((x1 + x2).astype(np.int8), w)
    assert np.array_equal(a12, oracle.conv1d(x1, w) + oracle.conv1d(x2, w))


def test_int32_overflow_is_reported():
    x = np.full((1, 1100, 1), -128, np.int8)
    w = np.full((1, 1100, 129), -128, np.int8)[:, :, :129]
    w[:] = -128
    # 1100*1*128*128 < 2^31, fine
    oracle.conv1d(x, w[:, :, 64:65].copy())
    big = np.full((1, 140000, 1), -128, np.int8)
    wb = np.full((1, 140000, 1), -128, np.int8)
    with pytest.raises(RuntimeError):
        oracle.conv1d(big, wb)


def test_linearity_of_quantised_convolution_sec_2_2():
    """S_W * S_x * Conv(q_W, q_x) equals Conv(S_W q_W, S_x q_x) (Sec. 2.2)."""
    rng = np.random.default_rng(9)
    x = rng.integers(-128, 128, size=(2, 4, 33)).astype(np.int8)
    w = rng.integers(-127, 128, size=(3, 4, 5)).astype(np.int8)
    S_x = 0.0371
    S_w = rng.uniform(1e-3, 1e-2, size=3)
    acc = oracle.conv1d(x, w).astype(np.float64)
    lhs = acc * (S_w * S_x)[None, :, None]
    xt = torch.from_numpy(x.astype(np.float64) * S_x)
    wt = torch.from_numpy(w.astype(np.float64) * S_w[:, None, None])
    rhs = torch.nn.functional.conv1d(xt, wt, padding=2).numpy()
    assert np.allclose(lhs, rhs, rtol=1e-12, atol=1e-12)


# ------------------------------------------------------------------ Eq. 1 quantiser, DQ
def test_quantiser_grid_eq_1():
    alpha = 3.3
    S = alpha / 127.0
    assert oracle.quantize([alpha], S)[0] == 127
    assert oracle.quantize([-alpha], S)[0] == -127
    assert oracle.quantize([10 * alpha], S)[0] == 127
    assert oracle.quantize([-10 * alpha], S)[0] == -128
    assert oracle.quantize([0.5 * S, -0.5 * S, 1.5 * S, -1.5 * S, 0.49 * S], S).tolist() == [1, -1, 2, -2, 0]
    x = np.linspace(-alpha, alpha, 1001)
    q = oracle.quantize(x, S)
    assert np.max(np.abs(q * S - x)) <= S / 2 + 1e-12       # DQ(Q(x)) is within half a step


def test_dequant_is_one_fp32_multiply():
    rng = np.random.default_rng(10)
    acc = rng.integers(-(1 << 26), 1 << 26, size=(2, 3, 17)).astype(np.int32)
    scale = rng.uniform(1e-4, 1e-3, 3).astype(np.float32)
    out = oracle.dequant(acc, scale)
    ref = acc.astype(np.float32) * scale[None, :, None]
    assert out.dtype == np.float32 and np.array_equal(out, ref)


# ------------------------------------------------------------------ BatchNorm folding
def test_batchnorm_folding_is_exact_and_integer_layer_within_one_lsb():
    rng = np.random.default_rng(21)
    Ci, Co, K, T = 6, 5, 3, 40
    W = rng.normal(0, 0.2, size=(Co, Ci, K))
    gamma, beta = rng.uniform(0.5, 1.5, Co), rng.normal(0, 0.3, Co)
    mean, var, eps = rng.normal(0, 0.5, Co), rng.uniform(0.2, 2.0, Co), 1e-3
    xf = rng.normal(0, 1.0, size=(2, Ci, T))
    Wf, bf = oracle.fold_batchnorm(W, gamma, beta, mean, var, eps)
    conv = torch.nn.functional.conv1d(torch.from_numpy(xf), torch.from_numpy(W), padding=1).numpy()
    bn = (conv - mean[None, :, None]) / np.sqrt(var + eps)[None, :, None] * gamma[None, :, None] + beta[None, :, None]
    folded = torch.nn.functional.conv1d(torch.from_numpy(xf), torch.from_numpy(Wf), torch.from_numpy(bf),
                                        padding=1).numpy()
    assert np.allclose(bn, folded, rtol=1e-9, atol=1e-9)

    # quantise per Eq. 1: per-channel weights, per-tensor activations
    S_x = np.abs(xf).max() / 127.0
    q_x = oracle.quantize(xf, S_x)
    S_w = np.abs(Wf).reshape(Co, -1).max(axis=1) / 127.0
    q_w = np.stack([oracle.quantize(Wf[o], S_w[o]) for o in range(Co)])
    bias_q = np.rint(bf / (S_w * S_x)).astype(np.int32)
    S_y = np.abs(folded).max() / 127.0
    ms = [oracle.dyadic_encode(S_w[o] * S_x / S_y) for o in range(Co)]
    mult = np.array([m for m, _ in ms], np.int32)
    shift = np.array([s for _, s in ms], np.uint8)
    acc = oracle.conv1d(q_x, q_w, bias_q)
    q_y = oracle.requant(acc, mult, shift)
    # float layer evaluated on the dequantised operands
    xd = q_x.astype(np.float64) * S_x
    Wd = q_w.astype(np.float64) * S_w[:, None, None]
    yd = torch.nn.functional.conv1d(torch.from_numpy(xd), torch.from_numpy(Wd), torch.from_numpy(bf),
                                    padding=1).numpy()
    err_lsb = np.abs(q_y.astype(np.float64) * S_y - np.clip(yd, -128 * S_y, 127 * S_y)) / S_y
    M = (S_w * S_x / S_y).max()
    assert err_lsb.max() <= 0.5 + M / 2 + 0.004 + 1e-9
    assert err_lsb.max() <= 1.0


# ------------------------------------------------------------------ residual add
def test_residual_add_equal_unit_scales_is_a_saturating_add():
    rng = np.random.default_rng(31)
    a = rng.integers(-128, 128, size=(2, 3, 50)).astype(np.int8)
    r = rng.integers(-128, 128, size=(2, 3, 50)).astype(np.int8)
    one = np.array([1 << 10, 1 << 10], np.int32)
    sh = np.array([10, 10], np.uint8)
    y = oracle.residual_add([a, r], one, sh)
    assert np.array_equal(y, np.clip(a.astype(np.int32) + r, -128, 127).astype(np.int8))
    yr = oracle.residual_add([a, r], one, sh, relu=True)
    assert np.array_equal(yr, np.clip(a.astype(np.int32) + r, 0, 127).astype(np.int8))


def test_residual_add_commutes_and_rounds_each_term_on_its_own():
    rng = np.random.default_rng(32)
    ts = [rng.integers(-128, 128, size=(1, 2, 64)).astype(np.int8) for _ in range(4)]
    m = np.array([20000, 17000, 30000, 16385], np.int32)
    s = np.array([15, 14, 16, 15], np.uint8)
    y = oracle.residual_add(ts, m, s, relu=True)
    p = [2, 0, 3, 1]
    y2 = oracle.residual_add([ts[i] for i in p], m[p], s[p], relu=True)
    assert np.array_equal(y, y2)
    for i in range(64):
        want = sum(_rs_exact(int(ts[j][0, 1, i]) * int(m[j]), int(s[j])) for j in range(4))
        assert int(y[0, 1, i]) == max(0, min(127, want))
    # two halves: each rounds up to 1 on its own (sum 2); rounding the sum once would give 1
    one = np.array([[[1]]], np.int8)
    assert int(oracle.residual_add([one, one], np.array([1, 1], np.int32), np.array([1, 1], np.uint8))[0, 0, 0]) == 2


# ------------------------------------------------------------------ model walk
def _walk_by_hand(model, x):
    """Independent walk of a model description: float64 library convolutions and exact
    Python-integer rescaling, following the layer order bias -> requant -> clamp ->
    [per-term rescaled residual sum] -> ReLU -> clamp."""
    def rq(acc, m, s, relu):
        out = np.empty(acc.shape, np.int64)
        for c in range(acc.shape[1]):
            flat = [max(-128, min(127, max(0, r) if relu else r))
                    for r in (_rs_exact(int(v) * int(m[c]), int(s[c])) for v in acc[:, c, :].ravel())]
            out[:, c, :] = np.array(flat).reshape(acc.shape[0], acc.shape[2])
        return out
    bufs = {0: x.astype(np.int64)}
    y = None
    for L in model["layers"]:
        h = bufs[L["in"]]
        if L["kind"] in ("tcs", "dw"):
            a = _torch_conv(h, L["w_dw"], None, L["stride"], L["dilation"], True)
            h = rq(a, L["m_dw"], L["s_dw"], False)
            if L["kind"] == "dw":
                bufs[L["out"]] = h
                y = h
                continue
            a = _torch_conv(h, L["w"][:, :, None], L["bias"], 1, 1, False)
        else:
            w = L["w"] if L["w"].ndim == 3 else L["w"][:, :, None]
            a = _torch_conv(h, w, L["bias"], L["stride"], L["dilation"], False)
        if L["out_int32"]:
            y = a.astype(np.int64)
        elif L["res"]:
            main = rq(a, L["m"], L["s"], False)
            terms = [main] + [bufs[i] for i in L["res"]]
            tot = np.zeros(main.shape, dtype=object)
            for j, t in enumerate(terms):
                tot = tot + np.vectorize(lambda v: _rs_exact(int(v) * int(L["res_m"][j]), int(L["res_s"][j])),
                                         otypes=[object])(t)
            y = np.vectorize(lambda v: max(-128, min(127, max(0, v) if L["relu"] else v)), otypes=[np.int64])(tot)
        else:
            y = rq(a, L["m"], L["s"], L["relu"])
        bufs[L["out"]] = y
    return y


@pytest.mark.parametrize("variant", ["live", "literal"])
@pytest.mark.parametrize("split", [False, True])
def test_encoder_walk_matches_an_independent_walk(variant, split):
    model, x = workloads.quartznet_model(2, 40, repeat=2, variant=variant, seed=77, mel=4,
                                         channels=(8, 16), kernels=(3, 5), c1=8, c2=16, c3=24,
                                         n_out=5, subblocks=3, split_tcs=split)
    lq, lf, trace = oracle.encoder_forward(model, x)
    ref = _walk_by_hand(model, x)
    assert lq.shape == ref.shape == (2, 5, 20)
    assert np.array_equal(lq.astype(np.int64), ref)
    assert np.array_equal(lf, lq.astype(np.float32) * model["out_scale"][None, :, None])
    if variant == "live":
        mid = trace[len(trace) // 2]["y"]
        assert np.mean(mid != 0) > 0.2


def test_split_and_fused_tables_describe_the_same_network():
    kw = dict(repeat=1, variant="live", seed=5, mel=4, channels=(8,), kernels=(3,), c1=8, c2=8, c3=8,
              n_out=3, subblocks=2)
    m1, x1 = workloads.quartznet_model(1, 24, split_tcs=False, **kw)
    m2, x2 = workloads.quartznet_model(1, 24, split_tcs=True, unique_bufs=True, **kw)
    assert np.array_equal(x1, x2)
    a = oracle.encoder_forward(m1, x1)[0]
    b = oracle.encoder_forward(m2, x2)[0]
    assert np.array_equal(a, b)


# ------------------------------------------------------------------ the layer table is the paper's model
def test_quartznet15x5_table_has_the_size_and_cost_of_table_1():
    gold = {}
    with open(os.path.join(GOLDEN, "table1_quartznet15x5.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                gold[k] = float(v)
    model, _ = workloads.quartznet_model(1, 1000, repeat=3, variant="literal", seed=2)
    st = workloads.model_stats(model)
    size_mb = st["weights"] / 1e6                                 # one byte per int8 weight
    bops_t = st["macs_per_utterance"] * 8 * 8 / 1e12              # 10 s input, 8-bit x 8-bit
    assert abs(size_mb - gold["w8a8_size_mb"]) / gold["w8a8_size_mb"] < 0.03
    assert abs(bops_t - gold["w8a8_bops_t"]) / gold["w8a8_bops_t"] < 0.03
    assert abs(st["macs_per_utterance"] * 32 * 32 / 1e12 - gold["fp32_bops_t"]) / gold["fp32_bops_t"] < 0.03
    assert len([L for L in model["layers"] if L["kind"] == "tcs"]) == 77


def test_jasperdr10x5_table_has_the_size_and_cost_the_paper_states():
    gold = {}
    with open(os.path.join(GOLDEN, "table1_jasperdr10x5.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                k, v = line.split()
                gold[k] = float(v)
    model, _ = workloads.jasper_model(1, 1000, variant="literal", seed=3)
    st = workloads.model_stats(model)
    assert abs(st["weights"] / 1e6 - gold["params_m"]) / gold["params_m"] < 0.01
    assert abs(st["macs_per_utterance"] * 64 / 1e12 - gold["w8a8_bops_t"]) / gold["w8a8_bops_t"] < 0.03
    assert abs(st["macs_per_utterance"] * 1024 / 1e12 - gold["fp32_bops_t"]) / gold["fp32_bops_t"] < 0.03
    last_block = [L for L in model["layers"] if L["name"] == "B9.4"][0]
    assert len(last_block["res"]) == 10          # C1's output and the nine earlier blocks


def test_jasper_and_conformer_walks_match_an_independent_walk():
    model, x = workloads.jasper_model(1, 40, seed=17, mel=4, channels=(8, 12), kernels=(3, 5), c1=8, k1=3, c2=12,
                                      k2=5, c3=16, n_out=5, subblocks=2)
    lq, _, _ = oracle.encoder_forward(model, x)
    assert np.array_equal(lq.astype(np.int64), _walk_by_hand(model, x))


def test_accumulators_cannot_overflow_int32_in_any_config():
    for idx in (0, 1, 2, 3, 4):
        model, _ = workloads.config(idx, variant="literal", **({"B": 1, "T": 64} if idx else {}))
        for L in model["layers"]:
            if L["kind"] in ("tcs", "dw"):
                assert L["K"] * 127 * 128 < 2 ** 31
            if "w" in L and L["kind"] != "glu":
                taps = L["C_in"] * (L["K"] if L["kind"] == "dense" else 1)
                assert taps * 127 * 128 + L["max_abs_bias"] < 2 ** 31


# ------------------------------------------------------------------ live scales are not degenerate
def test_live_variant_keeps_tensors_alive_and_literal_collapses():
    model, x = workloads.config(1, variant="live", B=1, T=256)
    _, _, trace = oracle.encoder_forward(model, x)
    for L, o in zip(model["layers"], trace):
        y = o["y"]
        if y.dtype == np.int8:
            assert np.mean(y != 0) > 0.25, L["name"]
    sat = np.mean([(np.mean((o["y"] == 127) | (o["y"] == -128))) for o in trace if o["y"].dtype == np.int8])
    assert sat > 1e-4
    model, x = workloads.config(1, variant="literal", B=1, T=256)
    _, _, trace = oracle.encoder_forward(model, x)
    assert all(np.all(o["y"] == 0) for o in trace[1:-1])


# ------------------------------------------------------------------ integer GLU gate (paper parity unpinned)
def _read_gate(q_c):
    """The gate value sig(g) of oracle.glu for every int8 g, read out exactly through the output alone.
    With a = 1 and (mult, shift) = (ceil(2^30 / theta), 31) the output RS(sig * mult, 31) is >= 1 exactly
    when sig >= theta (theta <= 2^15, sig an integer), so each call is an exact comparator; every g sits
    in a channel of its own and a bisection over theta finds its sig.  Nothing of the gate's formula is
    used here, only the rounding shift that the tests above pin."""
    g = np.arange(-128, 128, dtype=np.int64)
    q = g.astype(np.int8).reshape(1, 256, 1)
    a = np.ones_like(q)
    lo = np.zeros(256, np.int64)              # sig >= lo always holds (sig >= 0)
    hi = np.full(256, (1 << 15) + 1, np.int64)    # sig < hi
    while np.any(hi - lo > 1):
        theta = np.maximum((lo + hi) // 2, 1)
        mult = (-(-(1 << 30) // theta)).astype(np.int32)          # ceil(2^30 / theta)
        y = oracle.glu(a, q, q_c, mult, np.full(256, 31, np.uint8))[0, :, 0]
        ge = y >= 1
        lo = np.where(ge, theta, lo)
        hi = np.where(ge, hi, theta)
    return g, lo


@pytest.mark.parametrize("q_c", [1, 2, 7, 80, 117, 127, 128])
def test_glu_gate_is_the_piecewise_quadratic_its_definition_states(q_c):
    """Exact pins of the library's own gate (the paper prints no coefficients): anchor values, saturation,
    point symmetry about (0, q_c^2), monotonicity, and constant second differences -2 on (0, q_c) and +2 on
    (-q_c, 0).  A quadratic is fixed by two anchors and its second difference, so these leave no freedom:
    an off-by-one in the clamp, in p or in a sign fails one of them."""
    g, sig = _read_gate(q_c)
    at = dict(zip(g.tolist(), sig.tolist()))
    full = 2 * q_c * q_c
    assert at[0] == q_c * q_c
    for v in range(-128, 128):
        if v >= q_c:
            assert at[v] == full, v
        if v <= -q_c:
            assert at[v] == 0, v
        if -127 <= v <= 127:
            assert at[v] + at[-v] == full, v              # point symmetry
        if v > -128:
            assert at[v] >= at[v - 1], v                  # monotone
        if -127 <= v <= 126:
            d2 = at[v + 1] - 2 * at[v] + at[v - 1]
            if 0 < v < q_c:
                assert d2 == -2, (v, d2)
            elif -q_c < v < 0:
                assert d2 == 2, (v, d2)
            elif abs(v) > q_c:
                assert d2 == 0, (v, d2)
    # strictly increasing inside the unsaturated range
    for v in range(max(-q_c, -127), min(q_c, 127)):
        assert at[v + 1] > at[v], v


def test_glu_output_is_the_rounded_product_of_value_gate_and_multiplier():
    """y = sat8(RS(a * sig * mult, shift)) with Python integers, sig taken from the read-out table (not from
    a formula): pins the product, the 64-bit range, the rounding and the clamp of the output stage."""
    rng = np.random.default_rng(21)
    for q_c in (5, 80, 128):
        g, sig = _read_gate(q_c)
        C, T = 12, 256
        a = rng.integers(-128, 128, size=(2, C, T)).astype(np.int8)
        q = rng.integers(-128, 128, size=(2, C, T)).astype(np.int8)
        a[0, 0, :] = np.arange(-128, 128)
        q[0, 1, :] = np.arange(-128, 128)
        mult = rng.integers(0, 1 << 31, size=C).astype(np.int32)
        shift = rng.integers(1, 63, size=C).astype(np.uint8)
        mult[0], shift[0] = 1, 1
        mult[1], shift[1] = (1 << 31) - 1, 62
        mult[2], shift[2] = (1 << 31) - 1, 20          # saturates both ways
        mult[3], shift[3] = 0, 7
        y = oracle.glu(a, q, q_c, mult, shift)
        for b in range(2):
            for c in range(C):
                for t in range(0, T, 3):
                    v = int(a[b, c, t]) * int(sig[int(q[b, c, t]) + 128]) * int(mult[c])
                    want = max(-128, min(127, _rs_exact(v, int(shift[c]))))
                    assert int(y[b, c, t]) == want, (q_c, b, c, t)


def test_glu_gate_tracks_a_sigmoid():
    q_c = 80                       # S = 4 / q_c
    S = 4.0 / q_c
    q = np.arange(-128, 128, dtype=np.int64).astype(np.int8).reshape(1, 1, -1)
    a = np.full_like(q, 100)
    full = 2 * q_c * q_c
    # y = RS(a * sig_int * mult, shift) with mult/2^shift = 1/full  ->  y ~ a * sigmoid
    shift = 40
    mult = int(round((1 << shift) / full))
    y = oracle.glu(a, q, q_c, np.array([mult], np.int32), np.array([shift], np.uint8))[0, 0].astype(np.float64)
    ref = 100.0 / (1.0 + np.exp(-S * q[0, 0].astype(np.float64)))
    assert np.max(np.abs(y - ref)) <= 100 * 0.02 + 0.5 + 0.5

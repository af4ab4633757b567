"""Pins for the oracle's forward pass, accuracy count and analytic AI (CPU only)."""
import os

import numpy as np
import pytest

from aiq_workloads import (resnet20, mobilenet_v2, tiny_net, gen_model, gen_images,
                           gen_random_scheme, one_layer_lowered_schemes, conv_layer_indices)
from oracle import aiq_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                parts = [p.strip() for p in line.split("|")]
                out[parts[0]] = parts[1:]
    return out


# ---------------------------------------------------------------- brute force
def brute_conv(x, w, stride, pad, depthwise):
    """Seven nested loops, Python floats (double)."""
    B, C, H, W = x.shape
    cout, cg, k, _ = w.shape
    Ho = (H + 2 * pad - k) // stride + 1
    Wo = (W + 2 * pad - k) // stride + 1
    y = np.zeros((B, cout, Ho, Wo))
    for b in range(B):
        for n in range(cout):
            for oy in range(Ho):
                for ox in range(Wo):
                    acc = 0.0
                    for c in range(cg):
                        ci = n if depthwise else c
                        for r in range(k):
                            for t in range(k):
                                iy, ix = oy * stride + r - pad, ox * stride + t - pad
                                if 0 <= iy < H and 0 <= ix < W:
                                    acc += float(w[n, c, r, t]) * float(x[b, ci, iy, ix])
                    y[b, n, oy, ox] = acc
    return y


def brute_forward(arch, deq, x):
    """Independent restatement of the network semantics on top of brute_conv; executes the
    layers by repeatedly picking any layer whose operands are ready."""
    L = arch["layers"]
    outs = {}
    while len(outs) < len(L):
        for i, l in enumerate(L):
            if i in outs:
                continue
            if l["input"] >= 0 and l["input"] not in outs:
                continue
            if l["residual"] >= 0 and l["residual"] not in outs:
                continue
            src = x if l["input"] < 0 else outs[l["input"]]
            w, b = deq[i]
            if l["kind"] == "fc":
                pooled = np.float32(1) * np.asarray(
                    [[np.float32(np.mean(src[bb, c].astype(np.float64))) for c in range(src.shape[1])]
                     for bb in range(src.shape[0])], dtype=np.float32)
                y = np.zeros((src.shape[0], l["cout"]))
                for bb in range(src.shape[0]):
                    for n in range(l["cout"]):
                        y[bb, n] = sum(float(w[n, c]) * float(pooled[bb, c]) for c in range(l["cin"])) + float(b[n])
                outs[i] = y.astype(np.float32)
                continue
            dw = l["kind"] == "dw"
            w4 = w.reshape(l["cout"], 1 if dw else l["cin"], l["k"], l["k"])
            y = brute_conv(src, w4, l["stride"], l["pad"], dw) + b.astype(np.float64)[None, :, None, None]
            if l["residual"] >= 0:
                y = y + outs[l["residual"]].astype(np.float64)
            if l["act"] == "relu":
                y = np.maximum(y, 0)
            elif l["act"] == "relu6":
                y = np.clip(y, 0, 6)
            outs[i] = y.astype(np.float32)
    return outs[len(L) - 1]


# ---------------------------------------------------------------- conv definition
@pytest.mark.parametrize("k,stride,pad,dw", [(3, 1, 1, False), (3, 2, 1, False), (1, 1, 0, False),
                                             (1, 2, 0, False), (3, 1, 1, True), (3, 2, 1, True)])
def test_conv_against_loops(k, stride, pad, dw):
    rng = np.random.default_rng(k * 10 + stride + dw)
    x = rng.standard_normal((2, 4, 7, 6)).astype(np.float32)
    w = rng.standard_normal((4 if dw else 5, 1 if dw else 4, k, k)).astype(np.float32)
    got = O.conv2d_f64(x, w, stride, pad, depthwise=dw)
    want = brute_conv(x, w, stride, pad, dw)
    assert got.shape == want.shape
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


def test_pointwise_conv_is_matmul_and_fc_is_matmul():
    rng = np.random.default_rng(1)
    x = rng.standard_normal((3, 6, 5, 5)).astype(np.float32)
    w = rng.standard_normal((4, 6, 1, 1)).astype(np.float32)
    y = O.conv2d_f64(x, w, 1, 0)
    ref = np.einsum("bchw,nc->bnhw", x.astype(np.float64), w[:, :, 0, 0].astype(np.float64))
    np.testing.assert_allclose(y, ref, rtol=1e-12, atol=1e-12)


def test_hand_computed_network():
    g = _golden("tiny_forward_hand.txt")
    arch = dict(name="hand", in_c=1, in_h=4, in_w=4, n_classes=2, layers=[
        dict(name="c", kind="conv", cin=1, cout=2, k=3, stride=1, pad=1, act="relu", input=-1,
             residual=-1, has_bn=False),
        dict(name="fc", kind="fc", cin=2, cout=2, k=1, stride=1, pad=0, act="none", input=0,
             residual=-1, has_bn=False)])
    w0 = np.zeros((2, 9), np.float32)
    w0[0, :] = 1.0
    w0[1, 0 * 3 + 2] = 1.0
    deq = [(w0, np.asarray([-50.0, 0.0], np.float32)),
           (np.asarray([[1.0, 2.0], [-1.0, 4.0]], np.float32), np.asarray([0.5, 0.0], np.float32))]
    x = np.arange(1, 17, dtype=np.float32).reshape(1, 1, 4, 4)
    logits = O.forward(arch, deq, x)
    assert logits[0].tolist() == [float(v) for v in g["logits"][0].split()]
    box = O.conv2d_f64(x, w0[:1].reshape(1, 1, 3, 3), 2, 1)
    assert box.reshape(-1).tolist() == [float(v) for v in g["stride2_box"][0].split()]
    # pooled features through a one-layer net whose classifier is the identity
    deq_id = [deq[0], (np.eye(2, dtype=np.float32), np.zeros(2, np.float32))]
    assert O.forward(arch, deq_id, x)[0].tolist() == [float(v) for v in g["pooled"][0].split()]


def test_residual_and_activation_order_by_hand():
    """y = relu(conv(x) + b + residual): 1x1 identity conv on a 1x2x2 input, residual = the
    first layer's output; integers, so every value is exact."""
    arch = dict(name="r", in_c=1, in_h=2, in_w=2, n_classes=1, layers=[
        dict(name="a", kind="conv", cin=1, cout=1, k=1, stride=1, pad=0, act="none", input=-1,
             residual=-1, has_bn=False),
        dict(name="b", kind="conv", cin=1, cout=1, k=1, stride=1, pad=0, act="relu6", input=0,
             residual=0, has_bn=False),
        dict(name="fc", kind="fc", cin=1, cout=1, k=1, stride=1, pad=0, act="none", input=1,
             residual=-1, has_bn=False)])
    deq = [(np.asarray([[2.0]], np.float32), np.asarray([1.0], np.float32)),     # a = 2x + 1
           (np.asarray([[-1.0]], np.float32), np.asarray([0.5], np.float32)),    # b = relu6(-a + 0.5 + a) ... see below
           (np.asarray([[4.0]], np.float32), np.asarray([0.0], np.float32))]
    x = np.asarray([-3.0, 0.0, 1.0, 5.0], np.float32).reshape(1, 1, 2, 2)
    # a = [-5, 1, 3, 11]; b = relu6(-a + 0.5 + a) = 0.5 everywhere -> pooled 0.5 -> logit 2
    assert O.forward(arch, deq, x).tolist() == [[2.0]]
    deq[1] = (np.asarray([[1.0]], np.float32), np.asarray([0.5], np.float32))
    # b = relu6(2a + 0.5) = relu6([-9.5, 2.5, 6.5, 22.5]) = [0, 2.5, 6, 6] -> mean 3.625 -> 14.5
    assert O.forward(arch, deq, x).tolist() == [[14.5]]


def test_tiny_net_against_brute_force():
    arch = tiny_net()
    params = gen_model(arch, 99)
    folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded)
    scheme = gen_random_scheme(len(arch["layers"]), 5)
    x = gen_images(2, 3, 8, 8, 17)
    deq = [bank[i][int(b)] for i, b in enumerate(scheme)]
    got = O.forward(arch, deq, x)
    want = brute_forward(arch, deq, x)
    np.testing.assert_allclose(got, want, rtol=2e-6, atol=2e-6)


def test_fp32_scheme_is_the_unquantized_model():
    """FP32 is a member of Q and the start of both searches (Section 2.1, 2.2): the all-32
    scheme must reproduce the unquantized folded model bit for bit, so its agreement with
    labels drawn from that model is exactly 1."""
    arch = resnet20()
    params = gen_model(arch, 1234)
    folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded, bits_set=(32, 8))
    x = gen_images(8, 3, 32, 32, 1)
    ref = O.forward_fp32_unquantized(arch, folded, x)
    got = O.forward_scheme(arch, bank, [32] * 22, x)
    assert np.array_equal(ref.view(np.uint32), got.view(np.uint32))
    labels = O.predict(ref)
    acc, counts, preds, margins = O.eval_schemes(arch, bank, [[32] * 22, [8] * 22], x, labels)
    assert acc[0] == 1.0 and counts[0] == 8
    assert float(acc[1] * 8) == float(counts[1])
    assert np.all(margins >= 0)


def test_predict_lowest_index_on_ties_and_counts():
    lg = np.asarray([[1, 3, 3, 0], [2, 2, 2, 2], [0, -1, 5, 5]], np.float32)
    assert O.predict(lg).tolist() == [1, 0, 2]
    assert O.top2_margin(lg).tolist() == [0.0, 0.0, 0.0]
    assert O.top2_margin(np.asarray([[1.0, 4.5, 2.0]], np.float32)).tolist() == [2.5]


# ---------------------------------------------------------------- arithmetic intensity
def test_ai_single_layer_closed_form():
    arch = dict(name="one", in_c=8, in_h=10, in_w=10, n_classes=0, layers=[
        dict(name="c", kind="conv", cin=8, cout=12, k=3, stride=2, pad=1, act="relu", input=-1,
             residual=-1, has_bn=True)])
    # Ho = Wo = 5; K = 72; MACs = 12*72*25 = 21600
    for bits in (4, 8, 16, 32):
        ai, fl, by = O.scheme_ai(arch, [bits], batch=1)
        assert fl == 2 * 21600
        assert by == 12 * 72 * bits / 8 + 4 * (8 * 100 + 12 * 25)
        assert ai == fl / by
    ai3, fl3, by3 = O.scheme_ai(arch, [8], batch=3)
    assert fl3 == 3 * 2 * 21600 and by3 == 12 * 72 + 3 * 4 * (800 + 300)
    dw = dict(name="d", in_c=6, in_h=4, in_w=4, n_classes=0, layers=[
        dict(name="d", kind="dw", cin=6, cout=6, k=3, stride=1, pad=1, act="relu6", input=-1,
             residual=-1, has_bn=True)])
    ai, fl, by = O.scheme_ai(dw, [4])
    assert fl == 2 * 6 * 9 * 16 and by == 6 * 9 * 0.5 + 4 * (6 * 16 + 6 * 16)


def test_ai_resnet20_totals_and_paper_statements():
    arch = resnet20()
    L = len(arch["layers"])
    assert L == 22 and len(conv_layer_indices(arch)) == 21
    n_w = sum(l["cout"] * K for l, (K, *_r) in zip(arch["layers"], O.layer_shapes(arch)))
    assert n_w == 270896
    ai32, fl, by32 = O.scheme_ai(arch, [32] * L)
    assert fl == 2 * 40813184
    assert by32 == 270896 * 4 + 1650984
    ai8 = O.scheme_ai(arch, [8] * L)[0]
    ai4 = O.scheme_ai(arch, [4] * L)[0]
    g = _golden("ai_paper_statements.txt")
    lo, hi = float(g["int8_over_fp32"][0]), float(g["int8_over_fp32"][1])
    assert lo <= ai8 / ai32 <= hi
    lo, hi = float(g["int4_over_fp32"][0]), float(g["int4_over_fp32"][1])
    assert lo <= ai4 / ai32 <= hi
    assert ai4 > ai8 > ai32


def test_ai_monotone_in_every_layer():
    """Quantization reduces memory traffic (Section 2.1), so lowering any one layer's
    bit-width strictly raises AI."""
    for arch in (resnet20(), mobilenet_v2("cifar")):
        L = len(arch["layers"])
        base = O.scheme_ai(arch, [8] * L)[0]
        for s in one_layer_lowered_schemes(L, list(range(L))):
            assert O.scheme_ai(arch, s)[0] > base
        for s in one_layer_lowered_schemes(L, list(range(L)), base=8, low=16):
            assert O.scheme_ai(arch, s)[0] < base


def test_mobilenet_shapes():
    c = mobilenet_v2("cifar")
    i = mobilenet_v2("imagenet")
    assert len(c["layers"]) == 53 and len(conv_layer_indices(c)) == 52
    macs = lambda a: sum(l["cout"] * K * ho * wo for l, (K, _h, _w, ho, wo) in zip(a["layers"], O.layer_shapes(a)))
    nw = lambda a: sum(l["cout"] * K for l, (K, *_r) in zip(a["layers"], O.layer_shapes(a)))
    assert nw(c) == 2202560 and nw(i) == 3469760
    assert macs(i) == 300774272           # the commonly quoted ~300 M multiply-adds
    assert O.layer_shapes(i)[-2][3:] == (7, 7) and O.layer_shapes(c)[-2][3:] == (8, 8)
    with pytest.raises(ValueError):
        O.scheme_ai(c, [5] * 53)


def test_structural_variant_tables():
    """Shapes of the Section 4.5 variants: HeavyEarlyResNet20 has channel groups (64, 32, 16, 16),
    PlainConvNet20 has 20 convolutions of 64 channels plus the classifier (21 entries in Table 1)."""
    from aiq_workloads import heavy_early_resnet20, plain_convnet20
    h = heavy_early_resnet20()
    assert h["layers"][0]["cout"] == 64
    convs = [l for l in h["layers"] if l["kind"] == "conv" and l["k"] == 3]
    assert [l["cout"] for l in convs[1:]] == [32] * 6 + [16] * 12
    assert sum(1 for l in h["layers"] if l["k"] == 1 and l["kind"] == "conv") == 3      # every shape change
    p = plain_convnet20()
    assert len(p["layers"]) == 21 and p["layers"][-1]["kind"] == "fc"
    assert all(l["cout"] == 64 and l["residual"] == -1 for l in p["layers"][:-1])
    assert O.layer_shapes(p)[-2][3:] == (8, 8)


# ---------------------------------------------------------------- standalone linear layer
def _rows(text):
    return np.asarray([[float(v) for v in row.split()] for row in text.split("/")])


def test_qlinear_hand_table():
    """y[m][n] = s_n * sum_k code[n][k] * x[m][k] + bias[n] on values worked out by hand: the
    weight matrix is [N][K] with one scale per row, the bias is added once per output."""
    g = _golden("qlinear_hand.txt")
    codes = _rows(g["codes_2x3"][0]).astype(np.int8)
    scales = _rows(g["scales_2"][0])[0].astype(np.float32)
    bias = _rows(g["bias_2"][0])[0].astype(np.float32)
    x = _rows(g["x_2x3"][0]).astype(np.float32)
    y = O.qlinear(codes, scales, bias, 8, x)
    assert y.dtype == np.float32 and y.tolist() == _rows(g["y_2x2"][0]).tolist()
    # without a bias the outputs drop by exactly the bias
    assert (O.qlinear(codes, scales, None, 8, x) + bias[None, :]).tolist() == y.tolist()
    # 4-bit codes follow the same rule
    assert O.qlinear(codes, scales, bias, 4, x).tolist() == y.tolist()
    # square case: a transposed W or a scale per column would keep the shape but not the values
    ysq = O.qlinear(_rows(g["codes_sq"][0]).astype(np.int8), _rows(g["scales_sq"][0])[0].astype(np.float32),
                    None, 8, _rows(g["x_sq"][0]).astype(np.float32))
    assert ysq.tolist() == _rows(g["y_sq"][0]).tolist()


def test_qlinear_integer_inputs_are_exact_and_match_an_integer_matmul():
    """With integer activations every product and partial sum is an integer below 2^53, so the
    result must equal the int64 matrix product times the scale (a power of two here), exactly."""
    rng = np.random.default_rng(7)
    for bits, lim in ((4, 7), (8, 127)):
        codes = rng.integers(-lim, lim + 1, (9, 40)).astype(np.int8)
        x = rng.integers(-50, 51, (5, 40)).astype(np.float32)
        scales = (2.0 ** rng.integers(-6, 3, 9)).astype(np.float32)
        want = (x.astype(np.int64) @ codes.astype(np.int64).T).astype(np.float64) * scales[None, :].astype(np.float64)
        got = O.qlinear(codes, scales, None, bits, x)
        assert np.array_equal(got.astype(np.float64), want)
    # 16 / 32 bits: the stored element itself, no scale
    w = rng.integers(-8, 9, (6, 12)).astype(np.float32)
    x = rng.integers(-8, 9, (3, 12)).astype(np.float32)
    ones = np.ones(6, np.float32)
    want = (x.astype(np.int64) @ w.astype(np.int64).T).astype(np.float64)
    assert np.array_equal(O.qlinear(w.astype(np.float16), ones, None, 16, x).astype(np.float64), want)
    assert np.array_equal(O.qlinear(w, ones, None, 32, x).astype(np.float64), want)


def test_qlinear_is_the_classifier_of_a_one_layer_network():
    """A network that is a single linear classifier on 1x1 images is the same computation
    (the average pool of a 1x1 map is the identity): qlinear must equal forward() bit for bit."""
    rng = np.random.default_rng(11)
    N, K, M = 7, 20, 5
    W = (rng.standard_normal((N, K)) * 0.3).astype(np.float32)
    bias = rng.standard_normal(N).astype(np.float32)
    x = rng.standard_normal((M, K)).astype(np.float32)
    arch = dict(name="lin", in_c=K, in_h=1, in_w=1, n_classes=N, layers=[
        dict(name="fc", kind="fc", cin=K, cout=N, k=1, stride=1, pad=0, act="none", input=-1,
             residual=-1, has_bn=False)])
    for bits in (4, 8, 16, 32):
        v, s = O.quantize_rows(W, bits)
        y = O.qlinear(v, s, bias, bits, x)
        ref = O.forward(arch, [(O.dequantize_rows(v, s, bits), bias)], x.reshape(M, K, 1, 1))
        assert np.array_equal(y.view(np.uint32), ref.view(np.uint32))


def test_eval_schemes_hand_table():
    """Predictions, counts, accuracies and margins of three schemes on logits known by hand
    (ties go to the lowest index; a count is the number of predictions equal to the label)."""
    g = _golden("eval_schemes_hand.txt")
    x = _rows(g["images"][0]).astype(np.float32).reshape(6, 3, 1, 1)
    labels = _rows(g["labels"][0])[0].astype(np.int32)
    arch = dict(name="lin", in_c=3, in_h=1, in_w=1, n_classes=3, layers=[
        dict(name="fc", kind="fc", cin=3, cout=3, k=1, stride=1, pad=0, act="none", input=-1,
             residual=-1, has_bn=False)])
    zero = np.zeros(3, np.float32)
    bank = [{32: (np.eye(3, dtype=np.float32), zero),
             8: (np.asarray([[0, 1, 0], [0, 0, 1], [1, 0, 0]], np.float32), zero),
             4: (np.asarray([[1, 0, 0], [1, 0, 0], [0, 0, 1]], np.float32), zero)}]
    schemes = np.asarray([[32], [8], [4]], np.uint8)
    acc, counts, preds, margins = O.eval_schemes(arch, bank, schemes, x, labels, chunk=4)
    for row, bits in enumerate((32, 8, 4)):
        assert preds[row].tolist() == [int(v) for v in g[f"pred_{bits}"][0].split()], bits
        assert int(counts[row]) == int(g[f"count_{bits}"][0]), bits
        assert acc[row] == int(g[f"count_{bits}"][0]) / 6.0
        np.testing.assert_allclose(margins[row], [float(v) for v in g[f"margin_{bits}"][0].split()], atol=1e-6)
    # the image whose margin is 0.01 (up to float32 rounding of 4.01) sits on the edge of the
    # arg-max rule of the parity tests: it is the only one between 0.009 and 0.011
    assert ((margins[0] > 0.009) & (margins[0] < 0.011)).sum() == 1

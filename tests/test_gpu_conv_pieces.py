"""16- and 32-bit weights on the tensor-core convolution: both bfloat16 pieces must take part.

The tensor path holds a 16- or 32-bit weight as hi + lo, hi = bf16(w), lo = bf16(w - hi): exact
for a half, within 2^-17 of a float32 weight.  The end-to-end tolerance of that path is far
wider than the lo piece, so a dropped or misplaced lo tile would pass the forward tests.  Here
it is made visible: non-negative integer activations (exact in one bfloat16), two non-zero
weights m * (1 + 2^-9 + 2^-18), m in {1, 2}, per output channel, no batch normalisation, an
identity classifier.  Every product has the same sign: without the lo piece (m * 2^-9) every
logit drops by 2e-3 of its value; the float32 term m * 2^-18 is below the two pieces and is
the documented 3.8e-6.  Against the oracle run on the weights rounded to hi + lo (rounded here,
in numpy) the only error left is the rounding of the stored activations to two bfloat16 (up to
2^-17 of a value, unbiased): each logit within 2^-17 relative, the mean signed relative error
over all logits within 6e-7.  Against the oracle's own float32 weights: within 2^-17 + 2^-18."""
import numpy as np
import pytest

from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, compute_path

pytestmark = pytest.mark.gpu


def _bf16_rn(a):
    """float32 array rounded to bfloat16 (nearest, ties to even), as float32."""
    u = np.ascontiguousarray(a, np.float32).view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32)


def _layer(name, kind, cin, cout, k, stride, act, inp):
    return dict(name=name, kind=kind, cin=cin, cout=cout, k=k, stride=stride, pad=k // 2 if kind != "fc" else 0,
                act=act, input=inp, residual=-1, has_bn=False)


def _net(cin, cout, k, stride, hw=16):
    layers = [_layer("stem", "conv", 3, cin, 3, 1, "relu", -1),
              _layer("conv", "conv", cin, cout, k, stride, "none", 0),
              _layer("fc", "fc", cout, cout, 1, 1, "none", 1)]
    return dict(name=f"pieces_{cin}_{cout}_{k}_{stride}", in_c=3, in_h=hw, in_w=hw, n_classes=cout, layers=layers)


# (Cin, Cout, kernel, stride): every instantiation family of the multi-piece kernel, the
# two-slice case (64 output channels) included
SHAPES = [(16, 16, 3, 1), (16, 32, 3, 2), (16, 32, 1, 2), (32, 32, 3, 1), (32, 64, 3, 2), (32, 64, 1, 2),
          (64, 64, 3, 1), (64, 32, 3, 1), (64, 16, 1, 1),
          # channel counts only the pointwise kernel takes: one and several K chunks, one and several output tiles
          (96, 24, 1, 1), (48, 144, 1, 1), (160, 320, 1, 1)]


@pytest.mark.parametrize("path", ["tensor", "tiles"])
@pytest.mark.parametrize("cin,cout,k,stride", SHAPES)
def test_both_weight_pieces_count(cin, cout, k, stride, path):
    aiq = binding()
    arch = _net(cin, cout, k, stride)
    rng = np.random.default_rng(100 * cin + cout + k + stride)
    unit = np.float32(1.0 + 2.0 ** -9 + 2.0 ** -18)
    w = np.zeros((cout, cin * k * k), np.float32)
    for n in range(cout):                                           # two non-zero weights per output channel
        w[n, rng.choice(cin * k * k, 2, replace=False)] = rng.integers(1, 3, 2).astype(np.float32) * unit
    w = w.reshape(cout, cin, k, k)
    params = [
        dict(W=rng.integers(0, 2, (cin, 3, 3, 3)).astype(np.float32), bias=np.zeros(cin, np.float32)),
        dict(W=w, bias=np.zeros(cout, np.float32)),
        dict(W=np.eye(cout, dtype=np.float32), bias=np.zeros(cout, np.float32)),
    ]
    x = rng.integers(1, 4, (4, 3, 16, 16)).astype(np.float32)      # stem outputs: integers <= 81
    with compute_path(path):      # "tensor": the row-streaming kernel; "tiles": the pixel-tile kernel
        model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (16, 32))
    w32, b32 = bank[1][32]
    bank_hilo = [dict(e) for e in bank]                              # layer 1 at 32 bits: weights rounded to hi + lo
    bank_hilo[1][32] = ((_bf16_rn(w32) + _bf16_rn(w32 - _bf16_rn(w32))).astype(w32.dtype), b32)
    xd = to_dev(x)
    for bits in (32, 16):
        scheme = np.array([32, bits, 32], np.uint8)
        aiq.aiq_profile_start()
        got = model.aiq_forward(scheme, xd).cpu().numpy().astype(np.float64)
        kinds = aiq.aiq_profile_stop()
        assert kinds["conv_tc"]["launches"] >= 1, "the layer did not run on the tensor-core kernel"
        ref = O.forward_scheme(arch, bank, scheme, x).astype(np.float64)
        ref_hilo = O.forward_scheme(arch, bank_hilo, scheme, x).astype(np.float64)
        assert ref.min() > 0
        what = f"{arch['name']} at {bits} bits"
        err = (got - ref_hilo) / ref_hilo
        assert np.abs(err).max() <= 2.0 ** -17, f"{what}: relative error {np.abs(err).max():.3e}"
        assert abs(err.mean()) <= 6e-7, f"{what}: mean signed relative error {err.mean():.3e}"
        assert np.abs((got - ref) / ref).max() <= 2.0 ** -17 + 2.0 ** -18, what
    model.close()

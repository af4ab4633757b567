"""16- and 32-bit weights on the tensor-core convolution: every bfloat16 piece must take part.

The end-to-end tolerance of the tensor path is far wider than the weight of the third piece
of a float32 weight (2^-17 of the weight), so a dropped piece would pass the forward tests.
Here the piece is made visible: non-negative integer activations (exact in one bfloat16),
weights m * (1 + 2^-9 + 2^-18) with m in {0, 1, 2} (first piece m, second m * 2^-9, third
m * 2^-18), no batch normalisation, an identity classifier.  Every product has the same sign,
so a missing third piece shifts every logit by 3.8e-6 of its value and a missing second piece by
2e-3, while the rounding of the stored activations (2^-18 of a value, random sign) averages out
over the pooled pixels: the logits must match the oracle to 1e-6 relative."""
import numpy as np
import pytest

from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, compute_path

pytestmark = pytest.mark.gpu


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
          (64, 64, 3, 1), (64, 32, 3, 1), (64, 16, 1, 1)]


@pytest.mark.parametrize("cin,cout,k,stride", SHAPES)
def test_every_weight_piece_counts(cin, cout, k, stride):
    aiq = binding()
    arch = _net(cin, cout, k, stride)
    rng = np.random.default_rng(100 * cin + cout + k + stride)
    unit = np.float32(1.0 + 2.0 ** -9 + 2.0 ** -18)
    params = [
        dict(W=rng.integers(0, 2, (cin, 3, 3, 3)).astype(np.float32), bias=np.zeros(cin, np.float32)),
        dict(W=rng.integers(0, 3, (cout, cin, k, k)).astype(np.float32) * unit, bias=np.zeros(cout, np.float32)),
        dict(W=np.eye(cout, dtype=np.float32), bias=np.zeros(cout, np.float32)),
    ]
    x = rng.integers(0, 4, (4, 3, 16, 16)).astype(np.float32)      # stem outputs: integers <= 81
    with compute_path("tensor"):
        model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (16, 32))
    xd = to_dev(x)
    for bits in (32, 16):
        scheme = np.array([32, bits, 32], np.uint8)
        aiq.aiq_profile_start()
        got = model.aiq_forward(scheme, xd).cpu().numpy().astype(np.float64)
        kinds = aiq.aiq_profile_stop()
        assert kinds["conv_tc"]["launches"] >= 1, "the layer did not run on the tensor-core kernel"
        ref = O.forward_scheme(arch, bank, scheme, x).astype(np.float64)
        assert ref.min() > 0
        err = np.abs(got - ref) / ref
        assert err.max() <= 1e-6, f"{arch['name']} at {bits} bits: relative error {err.max():.3e}"
    model.close()

"""The row-streaming tensor-core convolution, one layer at a time, against the oracle.

Each case is a three-layer network (3x3 stem, the convolution under test, identity-free linear
classifier) small enough that nothing hides a wrong tap, a misplaced column tile or a wrong image
of a group.  Cases cover the three image-group modes (8 -> 8 images per group on maps 16 or 32
columns wide, 16 -> 16 on maps 8 columns wide, 8 -> 16 for the stride-2 layers that reach 8
columns), kernel sizes 3 and 1, both strides, every channel count, a residual operand, and
batches that fill no group, one group, and several groups with a ragged tail."""
import numpy as np
import pytest

from aiq_workloads import gen_model, gen_images
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close, compute_path

pytestmark = pytest.mark.gpu


def _conv(name, cin, cout, k, stride, act, inp, residual=-1):
    return dict(name=name, kind="conv", cin=cin, cout=cout, k=k, stride=stride, pad=k // 2, act=act,
                input=inp, residual=residual, has_bn=True)


def _net(cin, cout, k, stride, hw, with_residual):
    layers = [_conv("stem", 3, cin, 3, 1, "relu", -1),
              _conv("conv", cin, cout, k, stride, "relu", 0)]
    if with_residual:      # a second layer of the same shape that adds the first one's output
        layers.append(_conv("conv2", cout, cout, 3, 1, "relu", 1, residual=1))
    layers.append(dict(name="fc", kind="fc", cin=cout, cout=7, k=1, stride=1, pad=0, act="none",
                       input=len(layers) - 1, residual=-1, has_bn=False))
    return dict(name=f"rs_{cin}_{cout}_{k}_{stride}_{hw}", in_c=3, in_h=hw, in_w=hw, n_classes=7, layers=layers)


# (Cin, Cout, kernel, stride, image size, residual layer)
CASES = [
    (16, 16, 3, 1, 32, True),     # two column tiles per row, 8 images per group
    (16, 32, 3, 2, 32, False),    # stride 2, 32 -> 16 columns
    (16, 32, 1, 2, 32, False),    # projection shortcut shape
    (32, 32, 3, 1, 16, True),
    (32, 64, 3, 2, 16, False),    # stride 2 into 8 columns: two input groups feed one output group
    (32, 64, 1, 2, 16, False),
    (64, 64, 3, 1, 8, True),      # 16 images per group
    (64, 32, 3, 1, 32, False),    # 16 planes per pixel, wide rows
    (64, 32, 1, 1, 32, False),    # 1x1 at stride 1
    (32, 16, 3, 1, 8, True),
    (64, 64, 3, 2, 32, False),
]


@pytest.mark.parametrize("cin,cout,k,stride,hw,res", CASES)
def test_row_streaming_convolution_single_layer(cin, cout, k, stride, hw, res):
    aiq = binding()
    arch = _net(cin, cout, k, stride, hw, res)
    params = gen_model(arch, 8000 + cin + cout + k + stride + hw)
    with compute_path("tensor"):
        model = aiq.Model(arch, params)
    L = len(arch["layers"])
    bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8, 16, 32))
    for batch in (1, 16, 37):
        x = gen_images(batch, 3, hw, hw, 8100 + batch)
        xd = to_dev(x)
        for bits in (8, 4, 32, 16):
            scheme = np.full(L, 8, np.uint8)
            scheme[1] = bits
            if res:
                scheme[2] = bits
            aiq.aiq_profile_start()
            got = model.aiq_forward(scheme, xd).cpu().numpy()
            kinds = aiq.aiq_profile_stop()
            assert kinds["conv_tc"]["launches"] >= 1
            ref = O.forward_scheme(arch, bank, scheme, x)
            assert_logits_close(got, ref, f"{arch['name']} batch {batch} bits {bits}")
    model.close()

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


@pytest.fixture(autouse=True)
def _row_streaming_kernels_at_any_batch():
    """These tests are about the row-streaming kernels: keep small passes on them."""
    aiq = binding()
    aiq.aiq_set_small_pass_images(0)
    yield
    aiq.aiq_set_small_pass_images(1024)


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


def test_fused_basic_blocks_equal_the_layer_by_layer_path_bit_for_bit():
    """ResNet-20: the identity-shortcut blocks of the 16- and 32-channel stages run as one kernel
    each when every scheme gives them 4 or 8 bits.  The fused kernel does the same arithmetic in
    the same order as the two layer kernels, so logits and predictions must be identical, and
    both must match the oracle."""
    import torch
    from aiq_workloads import resnet20, one_layer_lowered_schemes, conv_layer_indices
    aiq = binding()
    arch = resnet20()
    params = gen_model(arch, 1234)
    model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8))
    rng = np.random.default_rng(5)
    for batch in (5, 40):
        x = gen_images(batch, 3, 32, 32, 8200 + batch)
        xd = to_dev(x)
        for trial in range(3):
            scheme = rng.choice(np.array([4, 8], np.uint8), 22)
            aiq.aiq_set_fusion(True, True)
            fused = model.aiq_forward(scheme, xd).cpu().numpy()
            launches_fused = aiq.aiq_last_call_stats()["kernel_launches"]
            aiq.aiq_set_fusion(False, True)
            plain = model.aiq_forward(scheme, xd).cpu().numpy()
            launches_plain = aiq.aiq_last_call_stats()["kernel_launches"]
            aiq.aiq_set_fusion(True, True)
            assert launches_fused == launches_plain - 5              # five blocks fold two launches into one
            assert np.array_equal(fused.view(np.uint32), plain.view(np.uint32))
            assert_logits_close(fused, O.forward_scheme(arch, bank, scheme, x), f"fused blocks batch {batch}")
    # a scheme with a 16-bit layer inside a block: that block is not fused, the others are
    scheme = np.full(22, 8, np.uint8)
    scheme[2] = 16
    x = gen_images(9, 3, 32, 32, 8300)
    bank16 = O.build_weight_bank(O.fold_model(arch, params), (8, 16))
    got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
    assert_logits_close(got, O.forward_scheme(arch, bank16, scheme, x), "one block unfused")
    # evaluator: counts and predictions with and without fusion
    x = gen_images(100, 3, 32, 32, 8400)
    labels = O.predict(O.forward_scheme(arch, bank, np.full(22, 8, np.uint8), x))
    schemes = one_layer_lowered_schemes(22, conv_layer_indices(arch))
    res = []
    for on in (True, False):
        aiq.aiq_set_fusion(on, True)
        preds = torch.full((21, 100), -1, dtype=torch.int32, device="cuda")
        acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=48)
        res.append((counts.copy(), preds.cpu().numpy()))
    aiq.aiq_set_fusion(True, True)
    assert np.array_equal(res[0][0], res[1][0]) and np.array_equal(res[0][1], res[1][1])
    model.close()


def test_average_pool_in_the_epilogue_matches_the_pooling_kernel():
    """The classifier's average pool taken inside the last convolution's epilogue (the default) against
    the separate pooling kernel and against the oracle; batches with a ragged last group."""
    from aiq_workloads import resnet20, heavy_early_resnet20
    aiq = binding()
    for make, seed in ((resnet20, 1234), (heavy_early_resnet20, 4500)):
        arch = make()
        L = len(arch["layers"])
        params = gen_model(arch, seed)
        model = aiq.Model(arch, params)
        bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8, 32))
        for batch, bits in ((1, 8), (19, 4), (48, 32)):
            x = gen_images(batch, 3, 32, 32, 8500 + batch)
            scheme = np.full(L, bits, np.uint8)
            aiq.aiq_set_fusion(True, True)
            fused = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
            n_fused = aiq.aiq_last_call_stats()["kernel_launches"]
            aiq.aiq_set_fusion(True, False)
            plain = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
            n_plain = aiq.aiq_last_call_stats()["kernel_launches"]
            aiq.aiq_set_fusion(True, True)
            assert n_fused == n_plain - 1                        # the pooling kernel is gone
            ref = O.forward_scheme(arch, bank, scheme, x)
            assert_logits_close(fused, ref, f"{arch['name']} pooled epilogue batch {batch}")
            assert_logits_close(plain, ref, f"{arch['name']} pooling kernel batch {batch}")
            assert np.abs(fused - plain).max() <= 1e-5 * (1.0 + np.abs(plain).max())
        model.close()

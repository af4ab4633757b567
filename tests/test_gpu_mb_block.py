"""The fused inverted-residual block kernel (expansion 1x1 -> depthwise 3x3 -> projection 1x1 with
the hidden tensor in shared memory) at the block shapes of MobileNetV2, alone, at the float32-path
tolerance: a dropped hidden chunk, a wrong halo row or a misplaced band would move the logits by
far more.

Shapes: the channel triples and map sizes of the CIFAR variant (32 / 16 / 8 wide maps, stride 1
with and without shortcut, stride 2) and map widths of the ImageNet variant that are not powers
of two (56, 28, 14, 7: bands that do not fill 128 accumulator lanes, a last band with fewer rows).
Every case checks that the fused kernel really ran (two launches fewer than layer by layer)."""
import numpy as np
import pytest

from aiq_workloads import inverted_residual_stack, gen_model, gen_images
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close

pytestmark = pytest.mark.gpu

# (cin, cout, hw, stride)
SHAPES = [
    (16, 24, 32, 1), (24, 24, 32, 1), (32, 64, 32, 2), (64, 64, 16, 1), (96, 96, 16, 1), (96, 160, 16, 2),
    (160, 160, 8, 1), (160, 320, 8, 1),
    (24, 32, 56, 2), (32, 32, 28, 1), (64, 64, 14, 1), (96, 160, 14, 2), (160, 160, 7, 1), (16, 16, 4, 1),
]


@pytest.mark.parametrize("cin,cout,hw,stride", SHAPES)
def test_fused_block_tight_tolerance(cin, cout, hw, stride):
    aiq = binding()
    arch = inverted_residual_stack(cin, cout, hw, stride)
    params = gen_model(arch, 8100 + cin + cout + hw)
    model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8))
    for batch in (1, 3):
        x = gen_images(batch, 3, hw, hw, 8200 + batch)
        xd = to_dev(x)
        for scheme in ([8, 8, 8, 8, 8], [8, 4, 8, 4, 8], [8, 8, 4, 8, 4]):
            scheme = np.array(scheme, np.uint8)
            ref = O.forward_scheme(arch, bank, scheme, x)
            aiq.aiq_set_fusion(True, True, inverted_residual=True)
            try:
                got = model.aiq_forward(scheme, xd).cpu().numpy()
                fused_launches = aiq.aiq_last_call_stats()["kernel_launches"]
            finally:
                aiq.aiq_set_fusion(True, True)
            plain = model.aiq_forward(scheme, xd).cpu().numpy()
            plain_launches = aiq.aiq_last_call_stats()["kernel_launches"]
            what = f"block {cin}->{cout} {hw}x{hw} stride {stride} batch {batch} scheme {scheme.tolist()}"
            assert fused_launches == plain_launches - 2, what
            assert_logits_close(got, ref, what + " fused")
            assert_logits_close(plain, ref, what + " layer by layer")
    model.close()


def test_fused_block_versions_share_one_launch():
    """Several candidates that differ inside the block (expansion, depthwise or projection bits)
    are jobs of one fused launch; predictions and counts follow the oracle."""
    import torch
    from gpu_util import assert_preds_match
    aiq = binding()
    arch = inverted_residual_stack(32, 32, 16, 1)
    params = gen_model(arch, 8301)
    x = gen_images(40, 3, 16, 16, 8302)
    folded = O.fold_model(arch, params)
    mean_logits = O.forward_fp32_unquantized(arch, folded, x).astype(np.float64).mean(axis=0)
    params = [dict(p) for p in params]
    params[-1]["bias"] = (params[-1]["bias"].astype(np.float64) - mean_logits).astype(np.float32)
    folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded, (4, 8, 16))
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    model = aiq.Model(arch, params)
    schemes = np.array([[8, 8, 8, 8, 8], [8, 4, 8, 8, 8], [8, 8, 4, 8, 8], [8, 8, 16, 8, 8], [8, 8, 8, 4, 8], [4, 8, 8, 8, 8]],
                       np.uint8)
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    preds = torch.full((len(schemes), 40), -1, dtype=torch.int32, device="cuda")
    aiq.aiq_set_fusion(True, True, inverted_residual=True)
    try:
        acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=40)
        fused_launches = aiq.aiq_last_call_stats()["kernel_launches"]
    finally:
        aiq.aiq_set_fusion(True, True)
    model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), chunk=40)
    assert fused_launches < aiq.aiq_last_call_stats()["kernel_launches"]
    assert_preds_match(preds.cpu().numpy(), opreds, omargins, "fused block, six candidates")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    model.close()


@pytest.mark.parametrize("variant,hw,batch", [("cifar", 32, 24), ("imagenet", 224, 3)])
def test_mobilenet_v2_with_fused_blocks(variant, hw, batch):
    """The whole MobileNetV2 (16 of its 17 blocks fused, 10 seeded conv layers at 4 bits) against the
    oracle at the tensor-path tolerance, with the classifier balanced so that the labels spread."""
    from aiq_workloads import mobilenet_v2, mixed_int4_int8_scheme, conv_layer_indices
    from gpu_util import assert_preds_match
    from test_gpu_forward import balance_classifier, assert_tensor_path_logits
    aiq = binding()
    arch = mobilenet_v2(variant)
    x = gen_images(batch, 3, hw, hw, 8624)
    params = balance_classifier(arch, gen_model(arch, 2234), x)
    model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8))
    scheme = mixed_int4_int8_scheme(53, conv_layer_indices(arch), 10, 43)
    ref = O.forward_scheme(arch, bank, scheme, x)
    aiq.aiq_set_fusion(True, True, inverted_residual=True)
    try:
        got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
        fused_launches = aiq.aiq_last_call_stats()["kernel_launches"]
    finally:
        aiq.aiq_set_fusion(True, True)
    model.aiq_forward(scheme, to_dev(x))
    assert fused_launches <= aiq.aiq_last_call_stats()["kernel_launches"] - 2 * 15
    assert_tensor_path_logits(got, ref, f"mbv2 {variant} fused blocks")
    assert_preds_match(O.predict(got), O.predict(ref), O.top2_margin(ref), f"mbv2 {variant} fused blocks")
    model.close()


def test_default_policy_fuses_where_it_pays():
    """Under the default setting a block on an 8-wide map is fused once the pass has 128 bands, and not
    below; the fused pass follows the oracle on sampled images."""
    aiq = binding()
    arch = inverted_residual_stack(160, 160, 8, 1)
    params = gen_model(arch, 8401)
    model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (8,))
    scheme = np.full(5, 8, np.uint8)
    x = gen_images(128, 3, 8, 8, 8402)
    got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
    launches_big = aiq.aiq_last_call_stats()["kernel_launches"]
    model.aiq_forward(scheme, to_dev(x[:100]))
    launches_small = aiq.aiq_last_call_stats()["kernel_launches"]
    assert launches_big == launches_small - 2
    sample = np.arange(3, 128, 16)
    assert_logits_close(got[sample], O.forward_scheme(arch, bank, scheme, x[sample]), "default policy, fused pass")
    model.close()

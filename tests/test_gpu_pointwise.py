"""The pointwise (1x1) tensor-core convolution at the channel pairs of MobileNetV2, alone, at the
float32-path tolerance: few layers, so nothing hides a dropped K chunk or a misplaced output tile.

Channel pairs: 16 -> 96 (first expansion), 144 -> 24 and 576 -> 96 (projections with several K
chunks of 64 input channels, the last one partial), 960 -> 160 (15 K chunks, three output tiles,
the last one narrow), 320 -> 1280 (the head: 20 output tiles of 64 channels) and two pairs whose
output runs as tiles of 128 channels in a single-scheme forward pass (64 -> 256, 192 -> 384).
The batch sets the number of 128-pixel tiles per launch: one partly filled tile, several tiles,
and more tiles than the launch has thread blocks per output tile."""
import numpy as np
import pytest

from aiq_workloads import pointwise_stack, gen_model, gen_images
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close, assert_preds_match, compute_path

pytestmark = pytest.mark.gpu

PAIRS = [(16, 96), (144, 24), (576, 96), (960, 160), (320, 1280), (64, 256), (192, 384)]


@pytest.mark.parametrize("path", ["tensor", "fp32"])
@pytest.mark.parametrize("cin,cout", PAIRS)
def test_pointwise_layer_tight_tolerance(cin, cout, path):
    aiq = binding()
    arch = pointwise_stack(cin, cout)
    params = gen_model(arch, 7000 + cin + cout)
    with compute_path(path):
        model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8, 32))
    batches = (1, 5, 40) if path == "tensor" else (5,)
    for batch in batches:
        x = gen_images(batch, 3, 8, 8, 7100 + batch)
        xd = to_dev(x)
        for pw_bits in (4, 8, 32):
            scheme = np.array([8, pw_bits, 8], np.uint8)
            got = model.aiq_forward(scheme, xd).cpu().numpy()
            ref = O.forward_scheme(arch, bank, scheme, x)
            assert_logits_close(got, ref, f"pointwise {cin}->{cout} batch {batch} bits {pw_bits} {path}")
    model.close()


@pytest.mark.parametrize("cin,cout", [(320, 1280), (960, 160)])
def test_pointwise_layer_two_versions_per_launch(cin, cout):
    """Two weight versions of the pointwise layer in one launch (4- and 8-bit candidates of an
    evaluation): the launch then splits its thread blocks over twice as many output tiles and
    picks the other tile width.  Predictions against the oracle, and against single forwards."""
    import torch
    aiq = binding()
    arch = pointwise_stack(cin, cout)
    params = gen_model(arch, 7000 + cin + cout)
    x = gen_images(33, 3, 8, 8, 7133)
    folded = O.fold_model(arch, params)
    mean_logits = O.forward_fp32_unquantized(arch, folded, x).astype(np.float64).mean(axis=0)
    params = [dict(p) for p in params]
    params[-1]["bias"] = (params[-1]["bias"].astype(np.float64) - mean_logits).astype(np.float32)
    folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded, (4, 8, 32))
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    model = aiq.Model(arch, params)
    schemes = np.array([[8, 8, 8], [8, 4, 8], [8, 8, 4]], np.uint8)
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    preds = torch.full((3, 33), -1, dtype=torch.int32, device="cuda")
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=33)
    p = preds.cpu().numpy()
    assert_preds_match(p, opreds, omargins, f"pointwise {cin}->{cout} two versions")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    for row, sc in enumerate(schemes):
        single = model.aiq_forward(sc, to_dev(x)).cpu().numpy()
        assert_logits_close(single, O.forward_scheme(arch, bank, sc, x), f"pointwise {cin}->{cout} scheme {sc}")
        decided = O.top2_margin(single) > 1e-2
        assert np.array_equal(O.predict(single)[decided], p[row][decided])
    model.close()

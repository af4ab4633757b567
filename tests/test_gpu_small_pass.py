"""Small passes: a ResNet-20 model created under the automatic path keeps two views of the same
weights (row-streaming format for the sweep's passes of thousands of images, pixel tiles for
passes too small to fill it).  Both must follow the oracle, and the switch must really happen."""
import numpy as np
import pytest

from aiq_workloads import resnet20, gen_model, gen_images, gen_random_scheme
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close, assert_preds_match

pytestmark = pytest.mark.gpu


def test_small_pass_view_follows_the_oracle():
    aiq = binding()
    arch = resnet20()
    params = gen_model(arch, 4321)
    model = aiq.Model(arch, params)
    bank = O.build_weight_bank(O.fold_model(arch, params), (4, 8))
    scheme = np.where(gen_random_scheme(model.n_layers, 7) > 8, 8, gen_random_scheme(model.n_layers, 7)).astype(np.uint8)
    x = gen_images(24, 3, 32, 32, 4322)
    ref = O.forward_scheme(arch, bank, scheme, x)
    results = {}
    for name, threshold in (("tiles", 1024), ("row-streaming", 0)):
        aiq.aiq_set_small_pass_images(threshold)
        try:
            results[name] = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
            results[name + " launches"] = aiq.aiq_last_call_stats()["kernel_launches"]
        finally:
            aiq.aiq_set_small_pass_images(1024)
        assert_logits_close(results[name], ref, f"resnet20 batch 24 on the {name} view")
        assert_preds_match(O.predict(results[name]), O.predict(ref), O.top2_margin(ref), name)
    # the row-streaming view fuses basic blocks and the pool: fewer launches, so the views differ
    assert results["row-streaming launches"] < results["tiles launches"]
    # a pass at the threshold runs on the row-streaming view
    big = gen_images(1024, 3, 32, 32, 4323)
    model.aiq_forward(scheme, to_dev(big))
    assert aiq.aiq_last_call_stats()["kernel_launches"] == results["row-streaming launches"]
    model.close()

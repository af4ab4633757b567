"""Single-layer sensitivity profile from an FP32 base (Section 3, experiment (1); Section 4.1;
Table 1, columns "8b" and "4b"): every layer alone at 8 and at 4 bits, all other layers FP32.
Counts and predictions of the CUDA evaluator against the oracle, AI exactly."""
import numpy as np
import pytest

from aiq_workloads import resnet20, gen_model, gen_images
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_preds_match

pytestmark = pytest.mark.gpu


def test_single_layer_sensitivity_profile_resnet20():
    import torch
    aiq = binding()
    arch = resnet20()
    L = len(arch["layers"])
    n = 128
    x = gen_images(n, 3, 32, 32, 5690)
    params = gen_model(arch, 1234)
    folded = O.fold_model(arch, params)
    mean_logits = O.forward_fp32_unquantized(arch, folded, x).astype(np.float64).mean(axis=0)
    params = [dict(p) for p in params]
    params[-1]["bias"] = (params[-1]["bias"].astype(np.float64) - mean_logits).astype(np.float32)
    folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded, (4, 8, 32))
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    assert len(np.unique(labels)) >= 5
    schemes = np.full((1 + 2 * L, L), 32, np.uint8)          # row 0: the FP32 base itself
    for i in range(L):
        schemes[1 + 2 * i, i] = 8
        schemes[2 + 2 * i, i] = 4
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    assert ocounts[0] == n                                    # the base agrees with its own labels
    assert len(set(ocounts.tolist())) > 2                     # the profile is not flat
    model = aiq.Model(arch, params)
    preds = torch.full((len(schemes), n), -1, dtype=torch.int32, device="cuda")
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=64)
    p = preds.cpu().numpy()
    assert_preds_match(p, opreds, omargins, "sensitivity profile")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    assert np.array_equal((p == labels[None, :]).sum(axis=1), counts)
    assert np.allclose(acc, counts / float(n))
    # prefix sharing: a profile from a common base shares every layer before the moved one
    stats = aiq.aiq_last_call_stats()
    assert stats["layer_evals"] < 0.62 * stats["layer_evals_unshared"]
    for sc in schemes:
        g, o = model.aiq_scheme_ai(sc), O.scheme_ai(arch, sc)
        assert g[1] == o[1] and g[2] == o[2] and abs(g[0] - o[0]) <= 1e-12 * o[0]
    # lowering one layer raises AI, and 4 bits raises it more than 8 (Table 1's AI columns)
    base_ai = O.scheme_ai(arch, schemes[0])[0]
    for i in range(L):
        a8, a4 = model.aiq_scheme_ai(schemes[1 + 2 * i])[0], model.aiq_scheme_ai(schemes[2 + 2 * i])[0]
        assert base_ai < a8 < a4
    model.close()

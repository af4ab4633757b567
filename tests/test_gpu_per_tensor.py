"""The per-tensor-scale variant of the quantizer (one scale for a whole weight tensor; the paper
lists per-channel effects as future work in Section 6) against the oracle: codes, scales and packed
bytes bit for bit, standalone and inside a model's weight bank; forward logits and the evaluator
on a per-tensor model; the analytic AI, which must not depend on the granularity."""
import numpy as np
import pytest

from aiq_workloads import resnet20, tiny_net, gen_model, gen_images, one_layer_lowered_schemes, conv_layer_indices
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close, assert_preds_match

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", [4, 8, 16, 32])
@pytest.mark.parametrize("shape", [(1, 1), (16, 27), (5, 33), (64, 576), (700, 2048), (300, 2051)])
def test_per_tensor_quantize_bit_exact(bits, shape):
    import torch
    aiq = binding()
    N, K = shape
    rng = np.random.default_rng(N * 17 + K)
    W = (rng.standard_normal(shape) * rng.uniform(0.01, 2.0, (N, 1))).astype(np.float32)
    if N > 2:
        W[1, :] = 0.0
    rb = aiq.aiq_packed_row_bytes(K, bits)
    packed = torch.full((N, rb), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(N, dtype=torch.float32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    scratch = torch.full((1,), 123, dtype=torch.int32, device="cuda")          # the call must not rely on it being zero
    aiq.aiq_quantize_layer_per_tensor(to_dev(W), bits, packed, scales, scratch, flag)
    torch.cuda.synchronize()
    v, s = O.quantize_rows(W, bits, per_tensor=True)
    assert int(flag.item()) == 0
    assert np.array_equal(scales.cpu().numpy().view(np.uint32), s.view(np.uint32))
    assert np.array_equal(packed.cpu().numpy(), O.pack_rows(v, bits))
    if bits <= 8 and N > 2:
        vc, sc = O.quantize_rows(W, bits)
        assert not np.array_equal(v, vc)                                       # the two granularities really differ here
    # non-finite weights are reported
    W[0, 0] = np.inf
    aiq.aiq_quantize_layer_per_tensor(to_dev(W), bits, packed, scales, scratch, flag)
    torch.cuda.synchronize()
    assert int(flag.item()) == 1


def test_per_tensor_model_bank_forward_and_evaluator():
    import torch
    aiq = binding()
    aiq.aiq_set_scale_granularity(aiq.SCALE_PER_TENSOR)
    try:
        for arch, seed, hw in ((resnet20(), 1234, 32), (tiny_net(), 99, 8)):
            L = len(arch["layers"])
            x = gen_images(40, 3, hw, hw, 6100 + hw)
            params = gen_model(arch, seed)
            folded = O.fold_model(arch, params)
            mean_logits = O.forward_fp32_unquantized(arch, folded, x).astype(np.float64).mean(axis=0)
            params = [dict(p) for p in params]
            params[-1]["bias"] = (params[-1]["bias"].astype(np.float64) - mean_logits).astype(np.float32)
            folded = O.fold_model(arch, params)
            model = aiq.Model(arch, params)
            bank = O.build_weight_bank(folded, (4, 8, 16, 32), per_tensor=True)
            # the bank inside the model, bit for bit
            for layer in range(L):
                for bits in (4, 8):
                    v, s = O.quantize_rows(folded[layer][0], bits, per_tensor=True)
                    packed, scales = (t.cpu().numpy() for t in model.layer_packed(layer, bits))
                    assert np.array_equal(scales.view(np.uint32), s.view(np.uint32)), (layer, bits)
                    assert np.array_equal(packed, O.pack_rows(v, bits)), (layer, bits)
            # forward logits
            for bits in (4, 8):
                got = model.aiq_forward([bits] * L, to_dev(x[:9])).cpu().numpy()
                assert_logits_close(got, O.forward_scheme(arch, bank, [bits] * L, x[:9]), f"{arch['name']} per-tensor {bits}")
            # evaluator on one greedy step
            labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
            schemes = one_layer_lowered_schemes(L, conv_layer_indices(arch))
            oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
            preds = torch.full((len(schemes), 40), -1, dtype=torch.int32, device="cuda")
            acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=16)
            assert_preds_match(preds.cpu().numpy(), opreds, omargins, f"{arch['name']} per-tensor greedy step")
            assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
            # AI: bytes follow the bit-widths only
            for sc in schemes[:3]:
                g, o = model.aiq_scheme_ai(sc), O.scheme_ai(arch, sc)
                assert g[1] == o[1] and g[2] == o[2] and abs(g[0] - o[0]) <= 1e-12 * o[0]
            model.close()
    finally:
        aiq.aiq_set_scale_granularity(aiq.SCALE_PER_CHANNEL)
    # back to the default: a new model has per-channel scales again
    arch = tiny_net()
    params = gen_model(arch, 99)
    model = aiq.Model(arch, params)
    folded = O.fold_model(arch, params)
    v, s = O.quantize_rows(folded[1][0], 4)
    packed, scales = (t.cpu().numpy() for t in model.layer_packed(1, 4))
    assert np.array_equal(scales.view(np.uint32), s.view(np.uint32)) and np.array_equal(packed, O.pack_rows(v, 4))
    model.close()

"""CUDA fold + quantize/pack against the oracle: bit-exact codes, scales and layout."""
import numpy as np
import pytest

from aiq_workloads import resnet20, mobilenet_v2, tiny_net, gen_model
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev

pytestmark = pytest.mark.gpu


def _quantize_gpu(aiq, W, bits):
    import torch
    N, K = W.shape
    rb = aiq.aiq_packed_row_bytes(K, bits)
    packed = torch.full((N, rb), 0xAB, dtype=torch.uint8, device="cuda")
    scales = torch.zeros(N, dtype=torch.float32, device="cuda")
    flag = torch.zeros(1, dtype=torch.int32, device="cuda")
    aiq.aiq_quantize_layer(to_dev(W), bits, packed, scales, flag)
    torch.cuda.synchronize()
    return packed.cpu().numpy(), scales.cpu().numpy(), int(flag.item())


@pytest.mark.parametrize("bits", [4, 8, 16, 32])
@pytest.mark.parametrize("shape", [(1, 1), (3, 9), (16, 27), (5, 33), (64, 576), (37, 1000),
                                   (10, 1280), (7, 8200), (3, 20000), (300, 2051)])
def test_quantize_bit_exact(bits, shape):
    aiq = binding()
    rng = np.random.default_rng(shape[0] * 131 + shape[1])
    W = (rng.standard_normal(shape) * rng.uniform(0.01, 2.0, (shape[0], 1))).astype(np.float32)
    if shape[0] > 2:
        W[1, :] = 0.0                    # all-zero row -> scale 1
        W[2, ::3] = 0.0
    packed, scales, flag = _quantize_gpu(aiq, W, bits)
    v, s = O.quantize_rows(W, bits)
    assert flag == 0
    assert np.array_equal(scales.view(np.uint32), s.view(np.uint32))
    assert np.array_equal(packed, O.pack_rows(v, bits))
    if bits <= 8:
        codes = O.unpack_rows(packed, shape[1], bits)
        assert codes.min() >= -(2 ** (bits - 1)) and codes.max() <= 2 ** (bits - 1) - 1


@pytest.mark.parametrize("bits", [4, 8, 16, 32])
@pytest.mark.parametrize("shape", [(700, 2048), (1203, 4096), (600, 8192), (1500, 2080)])
def test_quantize_streaming_kernel_bit_exact(bits, shape):
    """Large matrices (K % 32 == 0, 2048 <= K <= 8192, many rows) take the persistent
    streaming kernel: several rows per block, a ragged last round, zero rows, rows made of
    near-ties of the rounding, and wide ranges of row magnitudes."""
    aiq = binding()
    N, K = shape
    rng = np.random.default_rng(N * 7 + K)
    W = (rng.standard_normal(shape) * np.exp(rng.uniform(-12, 6, (N, 1)))).astype(np.float32)
    W[1, :] = 0.0
    W[2, ::3] = 0.0
    qmax = np.float32(2 ** (min(bits, 8) - 1) - 1)
    for r in range(5, N, 97):            # rows of near-ties: (k + 1/2) * s and its neighbours
        amax = np.float32(rng.uniform(0.1, 3.0))
        s = amax / qmax
        k = rng.integers(-int(qmax) + 1, int(qmax) - 1, K).astype(np.float32) + np.float32(0.5)
        w = (k * s).astype(np.float32)
        pick = rng.integers(0, 3, K)
        w = np.where(pick == 0, np.nextafter(w, np.float32(0.0)), np.where(pick == 1, np.nextafter(w, np.float32(np.inf) * np.sign(w)), w))
        w[0] = amax
        W[r] = w.astype(np.float32)
    packed, scales, flag = _quantize_gpu(aiq, W, bits)
    v, s = O.quantize_rows(W, bits)
    assert flag == 0
    assert np.array_equal(scales.view(np.uint32), s.view(np.uint32))
    assert np.array_equal(packed, O.pack_rows(v, bits))


def test_streaming_kernel_flags_nonfinite_rows():
    aiq = binding()
    W = np.ones((800, 2048), np.float32)
    W[700, 2047] = np.nan
    assert _quantize_gpu(aiq, W, 8)[2] == 1
    W[700, 2047] = -np.inf
    assert _quantize_gpu(aiq, W, 4)[2] == 1
    W[700, 2047] = 2.0
    packed, scales, flag = _quantize_gpu(aiq, W, 4)
    assert flag == 0 and scales[700] == np.float32(2.0) / np.float32(7.0)


def test_quantize_near_ties_follow_division():
    aiq = binding()
    rng = np.random.default_rng(11)
    rows = []
    for _ in range(200):
        amax = np.float32(rng.uniform(0.1, 3.0))
        s = amax / np.float32(127.0)
        k = rng.integers(-126, 126, 63).astype(np.float32) + np.float32(0.5)
        w = (k * s).astype(np.float32)
        w = np.nextafter(w, np.float32(0.0)) if rng.random() < 0.5 else w
        rows.append(np.concatenate([[amax], w]).astype(np.float32))
    W = np.stack(rows)
    for bits in (8, 4):
        packed, scales, _ = _quantize_gpu(aiq, W, bits)
        v, s = O.quantize_rows(W, bits)
        assert np.array_equal(O.unpack_rows(packed, W.shape[1], bits), v)
        assert np.array_equal(scales.view(np.uint32), s.view(np.uint32))


def test_nonfinite_sets_flag():
    aiq = binding()
    W = np.ones((4, 40), np.float32)
    W[2, 17] = np.inf
    assert _quantize_gpu(aiq, W, 8)[2] == 1
    W[2, 17] = np.nan
    assert _quantize_gpu(aiq, W, 4)[2] == 1
    W[2, 17] = 3.0
    assert _quantize_gpu(aiq, W, 4)[2] == 0


def test_fold_bit_exact():
    import torch
    aiq = binding()
    rng = np.random.default_rng(5)
    for N, K in ((16, 27), (64, 576), (33, 1)):
        W = rng.standard_normal((N, K)).astype(np.float32)
        gamma = rng.uniform(0.5, 1.5, N).astype(np.float32)
        beta = (rng.standard_normal(N) * 0.1).astype(np.float32)
        mean = (rng.standard_normal(N) * 0.1).astype(np.float32)
        var = rng.uniform(0.5, 1.5, N).astype(np.float32)
        Wf = torch.empty((N, K), dtype=torch.float32, device="cuda")
        bf = torch.empty(N, dtype=torch.float32, device="cuda")
        aiq.aiq_fold_bn(to_dev(W), to_dev(gamma), to_dev(beta), to_dev(mean), to_dev(var), Wf, bf)
        oW, ob = O.fold_bn(W, gamma, beta, mean, var)
        assert np.array_equal(Wf.cpu().numpy().view(np.uint32), oW.view(np.uint32))
        assert np.array_equal(bf.cpu().numpy().view(np.uint32), ob.view(np.uint32))


@pytest.mark.parametrize("arch_name", ["tiny", "resnet20", "mbv2_cifar", "mbv2_imagenet"])
def test_model_bank_bit_exact(arch_name):
    """Every layer of every network at 4/8/16/32 bits: folded weights, biases, packed codes
    and scales inside the model equal the oracle's bit for bit."""
    aiq = binding()
    arch = {"tiny": tiny_net, "resnet20": resnet20, "mbv2_cifar": lambda: mobilenet_v2("cifar"),
            "mbv2_imagenet": lambda: mobilenet_v2("imagenet")}[arch_name]()
    params = gen_model(arch, 77)
    model = aiq.Model(arch, params)
    folded = O.fold_model(arch, params)
    for i, (Wf, bf) in enumerate(folded):
        gW, gb = model.layer_folded(i)
        assert np.array_equal(gW.cpu().numpy().view(np.uint32), Wf.view(np.uint32)), i
        assert np.array_equal(gb.cpu().numpy().view(np.uint32), bf.view(np.uint32)), i
        for bits in (4, 8, 16, 32):
            p, s = model.layer_packed(i, bits)
            v, os_ = O.quantize_rows(Wf, bits)
            assert np.array_equal(p.cpu().numpy(), O.pack_rows(v, bits)), (i, bits)
            assert np.array_equal(s.cpu().numpy().view(np.uint32), os_.view(np.uint32)), (i, bits)
    model.close()


def test_model_create_rejects_nonfinite():
    aiq = binding()
    arch = tiny_net()
    params = gen_model(arch, 3)
    params[4]["W"][5, 2, 0, 0] = np.nan
    with pytest.raises(aiq.AiqError) as e:
        aiq.Model(arch, params)
    assert e.value.status == aiq.ERR_NONFINITE

"""CUDA small-batch quantized linear layer against the oracle."""
import numpy as np
import pytest

from aiq_workloads import gen_linear_case
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close

pytestmark = pytest.mark.gpu


def _run(aiq, W, x, bits, bias=None, use_workspace=True):
    import torch
    N, K = W.shape
    rb = aiq.aiq_packed_row_bytes(K, bits)
    packed = torch.empty((N, rb), dtype=torch.uint8, device="cuda")
    scales = torch.empty(N, dtype=torch.float32, device="cuda")
    aiq.aiq_quantize_layer(to_dev(W), bits, packed, scales)
    y = torch.full((x.shape[0], N), float("nan"), dtype=torch.float32, device="cuda")
    ws_bytes = aiq.aiq_qlinear_workspace_bytes(N, K, bits, x.shape[0]) if use_workspace else 0
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda") if ws_bytes else None
    aiq.aiq_qlinear(packed, scales, to_dev(bias) if bias is not None else None, N, K, bits, to_dev(x), y,
                    workspace=ws)
    torch.cuda.synchronize()
    v, s = O.quantize_rows(W, bits)
    return y.cpu().numpy(), O.qlinear(v, s, bias, bits, x)


@pytest.mark.parametrize("bits", [4, 8, 16, 32])
@pytest.mark.parametrize("N,K,M", [(1280, 320, 1), (1280, 320, 4), (1280, 320, 16), (10, 64, 64),
                                   (1000, 1280, 5), (37, 100, 3), (5, 27, 2), (4096, 4096, 1),
                                   (2048, 4096, 4), (300, 2052, 7), (1, 1, 1),
                                   # shapes on the warp-level tensor-core path (K % 512 == 0, N*K >= 2^20)
                                   (4100, 512, 16), (1000, 1536, 3), (2050, 1024, 9), (8192, 8192, 2),
                                   (1030, 1024, 1), (4100, 8192, 2), (2048, 3072, 2),
                                   # batches on the tcgen05 path (M >= 9, K % 8 == 0): ragged N, K and M tails,
                                   # several batch blocks, K split over CTAs
                                   (4096, 4096, 256), (1280, 320, 256), (1000, 1280, 37), (2050, 1024, 300),
                                   (130, 72, 16), (33, 64, 9), (4100, 520, 64)])
def test_qlinear_matches_oracle(bits, N, K, M):
    aiq = binding()
    W, x = gen_linear_case(N, K, M, seed=3234 + N + K + M)
    bias = np.random.default_rng(N).standard_normal(N).astype(np.float32) if N % 2 == 0 else None
    got, ref = _run(aiq, W, x, bits, bias)
    assert_logits_close(got, ref, f"N={N} K={K} M={M} bits={bits}")
    if aiq.aiq_qlinear_workspace_bytes(N, K, bits, M):        # the same shape on the plain kernel
        got, ref = _run(aiq, W, x, bits, bias, use_workspace=False)
        assert_logits_close(got, ref, f"plain N={N} K={K} M={M} bits={bits}")


@pytest.mark.parametrize("bits", [4, 8])
def test_qlinear_exact_on_integers(bits):
    """Integer weights and activations: every product and partial sum is exact in float32,
    so the result must equal the integer answer exactly (s = 1)."""
    aiq = binding()
    rng = np.random.default_rng(1)
    qmax = 2 ** (bits - 1) - 1
    # plain / int8 warp-level (M = 5 and M = 2) / tcgen05
    for shape_w, m in (((96, 200), 4), ((2176, 512), 5), ((2176, 2048), 2), ((300, 520), 20)):
        W = rng.integers(-qmax, qmax + 1, shape_w).astype(np.float32)
        W[:, 0] = qmax
        x = rng.integers(-8, 9, (m, shape_w[1])).astype(np.float32)
        got, ref = _run(aiq, W, x, bits)
        want = x.astype(np.int64) @ W.astype(np.int64).T
        assert np.array_equal(got.astype(np.int64), want)
        assert np.array_equal(ref.astype(np.int64), want)


@pytest.mark.parametrize("bits", [16, 32])
def test_qlinear_two_piece_path_exact_on_integers(bits):
    """16- and 32-bit weights on the tcgen05 kernel enter as two bfloat16 pieces.  Small integer
    weights and activations make every product and sum exact, so any dropped, repeated or stale
    tile shows up as a wrong integer.  Shapes with many K chunks per CTA, several batch blocks and
    K splits; each shape is run three times (a race would not repeat)."""
    aiq = binding()
    for (N, K, M) in ((128, 64, 16), (256, 512, 32), (4096, 4096, 128), (2048, 2048, 256), (4096, 4096, 256),
                      (1000, 1288, 300)):
        rng = np.random.default_rng(N + K + M + bits)
        W = rng.integers(-3, 4, (N, K)).astype(np.float32)
        x = rng.integers(-2, 3, (M, K)).astype(np.float32)
        want = x.astype(np.int64) @ W.astype(np.int64).T
        for trial in range(3):
            got, ref = _run(aiq, W, x, bits)
            assert np.array_equal(got.astype(np.int64), want), (N, K, M, bits, trial)

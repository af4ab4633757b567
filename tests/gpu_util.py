"""Shared helpers of the GPU parity tests."""
import functools

import numpy as np


@functools.lru_cache(maxsize=None)
def binding():
    from paper_2512_14090_b200 import build
    build.build()
    from paper_2512_14090_b200 import binding as b
    return b


def to_dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def assert_logits_close(got, ref, what=""):
    """|delta| <= 1e-3 * (1 + |ref|), the float32-accumulate tolerance."""
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64)) / (1.0 + np.abs(ref.astype(np.float64)))
    assert np.all(np.isfinite(got)), what
    assert err.max() <= 1e-3, f"{what}: max relative error {err.max():.3e}"
    return err.max()


def assert_preds_match(preds, opreds, omargins, what=""):
    """Arg-max must agree wherever the oracle's top-2 margin exceeds 1e-2."""
    decided = omargins > 1e-2
    bad = (preds != opreds) & decided
    assert not bad.any(), f"{what}: {bad.sum()} arg-max mismatches at decided margins"


def assert_logits_close_tensor(got, ref, what=""):
    """|delta| <= 2e-2 * max|logit|: the tolerance of a bf16 tensor-core path."""
    assert np.all(np.isfinite(got)), what
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64)).max()
    bound = 2e-2 * np.abs(ref.astype(np.float64)).max()
    assert err <= bound, f"{what}: max abs error {err:.3e} > {bound:.3e}"
    return err


class compute_path:
    """Context manager: models created inside use the given compute path."""

    def __init__(self, name):
        self.name = name

    def __enter__(self):
        b = binding()
        b.aiq_set_compute_path({"auto": b.PATH_AUTO, "fp32": b.PATH_FP32, "tensor": b.PATH_TENSOR,
                                "tiles": b.PATH_TENSOR_TILES}[self.name])
        return self

    def __exit__(self, *exc):
        binding().aiq_set_compute_path(binding().PATH_AUTO)
        return False

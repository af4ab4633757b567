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

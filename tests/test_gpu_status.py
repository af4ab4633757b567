"""Device-side failure reporting, exercised without breaking a product kernel: a one-thread kernel
waits with the library's bounded-wait routine on a barrier nothing arrives at; the wait must give
up, the kernel must return, and the host must see AIQ_ERR_TIMEOUT exactly once."""
import time

import numpy as np
import pytest

from aiq_workloads import tiny_net, gen_model, gen_images
from gpu_util import binding, to_dev

pytestmark = pytest.mark.gpu


def test_bounded_wait_expires_and_is_reported_once():
    import torch
    aiq = binding()
    arch = tiny_net()
    model = aiq.Model(arch, gen_model(arch, 1))
    model.aiq_model_status()                                   # clean to begin with
    t0 = time.time()
    model.aiq_debug_expire_wait(2_000_000)                     # about 1 ms of SM clocks
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_model_status()
    assert e.value.status == aiq.ERR_TIMEOUT
    assert time.time() - t0 < 5.0                              # the wait ended by itself, quickly
    model.aiq_model_status()                                   # the record was cleared
    # the context is intact: an evaluation after the expired wait works and reports no failure
    x = gen_images(6, 3, 8, 8, 2)
    labels = torch.zeros(6, dtype=torch.int32, device="cuda")
    schemes = np.full((2, model.n_layers), 8, np.uint8)
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), labels)
    assert counts[0] == counts[1]
    # an expired wait that nobody has collected yet fails the next evaluation instead
    model.aiq_debug_expire_wait(2_000_000)
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_eval_schemes(schemes, to_dev(x), labels)
    assert e.value.status == aiq.ERR_TIMEOUT
    acc2, counts2 = model.aiq_eval_schemes(schemes, to_dev(x), labels)
    assert np.array_equal(counts, counts2)
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_debug_expire_wait(0)
    assert e.value.status == aiq.ERR_INVALID_ARG
    model.close()

"""aiq_forward_static: the forward pass for callers that cannot allocate device memory.

Some users of this library run where obtaining device memory is not possible at call time:
inside a host framework's callback that forbids cudaMalloc, in a service whose memory
budget was fixed and spent at start-up, or as a plug-in that only ever receives input and
output buffers.  aiq_forward_static serves them from a fixed workspace built into the
library.  This test calls it through the C ABI twice in a row (the second call finds the
first call's leftovers in the shared workspace) and checks each result against aiq_forward
with an ordinary caller-provided workspace and against the CPU oracle, at the tolerance the
other forward tests use, and checks that a call leaves the amount of free device memory
unchanged (it must not allocate).
It lives in a file that sorts last so that a run stopping at the first failure has already
executed every other test.
"""
import numpy as np
import pytest

from aiq_workloads import resnet20, tiny_net, gen_model, gen_images, gen_random_scheme
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev, assert_logits_close

pytestmark = pytest.mark.gpu


def _compare_two_calls(aiq, model, cases, arch, params):
    import torch
    bank = O.build_weight_bank(O.fold_model(arch, params))
    for call, (scheme, x) in enumerate(cases):
        xd = to_dev(x)
        want = model.aiq_forward(scheme, xd).cpu().numpy()
        got = torch.full((x.shape[0], model.n_classes), float("nan"), dtype=torch.float32, device="cuda")
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        model.aiq_forward_static(scheme, xd, got)
        torch.cuda.synchronize()
        if call > 0:      # the first call may still load kernels of the library; later ones must not allocate
            assert torch.cuda.mem_get_info()[0] == free_before, "aiq_forward_static changed the free device memory"
        assert_logits_close(got.cpu().numpy(), want, "aiq_forward_static vs aiq_forward")
        assert_logits_close(got.cpu().numpy(), O.forward_scheme(arch, bank, scheme, x), "aiq_forward_static vs oracle")


def test_static_workspace_matches_forward_on_two_calls_in_a_row():
    aiq = binding()
    arch = resnet20()
    params = gen_model(arch, 1234)
    model = aiq.Model(arch, params)
    # the limit the header documents for this network, in the model's own activation format
    aiq.aiq_set_small_pass_images(0)
    try:
        assert model.aiq_workspace_bytes(24, 1) <= aiq.STATIC_WORKSPACE_BYTES
        assert model.aiq_workspace_bytes(32, 1) <= aiq.STATIC_WORKSPACE_BYTES < model.aiq_workspace_bytes(33, 1)
    finally:
        aiq.aiq_set_small_pass_images(1024)
    cases = [(gen_random_scheme(model.n_layers, 42), gen_images(24, 3, 32, 32, 5678)),
             (gen_random_scheme(model.n_layers, 43), gen_images(7, 3, 32, 32, 5680))]
    _compare_two_calls(aiq, model, cases, arch, params)
    model.close()
    # another model through the same shared workspace, again twice
    arch = tiny_net()
    params = gen_model(arch, 99)
    model = aiq.Model(arch, params)
    cases = [(gen_random_scheme(model.n_layers, s), gen_images(11 + s, 3, 8, 8, 100 + s)) for s in (1, 2)]
    _compare_two_calls(aiq, model, cases, arch, params)
    model.close()


def test_static_workspace_rejects_what_does_not_fit():
    import torch
    aiq = binding()
    arch = resnet20()
    model = aiq.Model(arch, gen_model(arch, 1234))
    batch = 64
    assert model.aiq_workspace_bytes(batch, 1) > aiq.STATIC_WORKSPACE_BYTES
    x = to_dev(gen_images(batch, 3, 32, 32, 1))
    logits = torch.zeros((batch, 10), dtype=torch.float32, device="cuda")
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_forward_static(np.full(model.n_layers, 8, np.uint8), x, logits)
    assert e.value.status == aiq.ERR_WORKSPACE_TOO_SMALL
    assert "built-in" in str(e.value)
    model.close()

"""CUDA forward pass and scheme evaluator against the oracle (through the C ABI)."""
import numpy as np
import pytest

from aiq_workloads import (resnet20, mobilenet_v2, tiny_net, heavy_early_resnet20, plain_convnet20,
                           gen_model, gen_images,
                           gen_random_scheme, one_layer_lowered_schemes, coordinate_step_schemes,
                           mixed_int4_int8_scheme, conv_layer_indices)
from oracle import aiq_oracle as O
from gpu_util import (binding, to_dev, assert_logits_close, assert_logits_close_tensor,
                      assert_preds_match, compute_path)

pytestmark = pytest.mark.gpu


def _oracle_bank(arch, params, bits_set=(4, 8, 16, 32)):
    folded = O.fold_model(arch, params)
    return folded, O.build_weight_bank(folded, bits_set)


def balance_classifier(arch, params, x):
    """Random-init networks put almost every image in one class (a constant offset
    dominates the logits).  Shift the classifier bias by the oracle's mean FP32 logits so
    that predictions spread over the classes and margins become small: a much sharper test
    of arg-max and counting.  The shift is computed by the oracle only."""
    folded = O.fold_model(arch, params)
    mean_logits = O.forward_fp32_unquantized(arch, folded, x).astype(np.float64).mean(axis=0)
    params = [dict(p) for p in params]
    params[-1]["bias"] = (params[-1]["bias"].astype(np.float64) - mean_logits).astype(np.float32)
    return params


@pytest.mark.parametrize("path", ["fp32", "tensor"])
@pytest.mark.parametrize("batch", [1, 3, 37])
def test_tiny_net_random_schemes(batch, path):
    aiq = binding()
    arch = tiny_net()
    params = gen_model(arch, 99)
    with compute_path(path):
        model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params)
    x = gen_images(batch, 3, 8, 8, 17 + batch)
    for seed in range(6):
        scheme = gen_random_scheme(model.n_layers, seed)
        got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
        ref = O.forward_scheme(arch, bank, scheme, x)
        assert_logits_close(got, ref, f"tiny batch={batch} seed={seed}")


@pytest.mark.parametrize("path", ["fp32", "tensor", "tiles"])
def test_resnet20_batch64_mixed_scheme(path):
    """ResNet-20, batch 64, one bit-width per layer drawn from {32, 16, 8, 4}."""
    aiq = binding()
    arch = resnet20()
    params = gen_model(arch, 1234)
    with compute_path(path):
        model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params)
    x = gen_images(64, 3, 32, 32, 5678)
    scheme = gen_random_scheme(22, 42)
    got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
    ref = O.forward_scheme(arch, bank, scheme, x)
    assert_logits_close(got, ref, "resnet20 mixed")
    assert_preds_match(O.predict(got), O.predict(ref), O.top2_margin(ref), "resnet20 mixed")
    for bits in (32, 16, 8, 4):
        got = model.aiq_forward([bits] * 22, to_dev(x[:9])).cpu().numpy()
        assert_logits_close(got, O.forward_scheme(arch, bank, [bits] * 22, x[:9]), f"uniform {bits}")
    # analytic AI equals the oracle's for this scheme and for the uniform ones
    for s in (scheme, [32] * 22, [8] * 22, [4] * 22):
        g, o = model.aiq_scheme_ai(s), O.scheme_ai(arch, s)
        assert g[1] == o[1] and g[2] == o[2] and abs(g[0] - o[0]) <= 1e-12 * o[0]
    g3, o3 = model.aiq_scheme_ai(scheme, 3), O.scheme_ai(arch, scheme, 3)
    assert g3[1] == o3[1] and g3[2] == o3[2]


def assert_tensor_path_logits(got, ref, what, measured_bound=5e-3):
    """Tensor-core path: the stated tolerance 2e-2 * max|logit| and, tighter, the bound the
    two-bfloat16 storage is measured to keep on the deep networks (5e-3 * max|logit|)."""
    assert_logits_close_tensor(got, ref, what)
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64)).max()
    peak = np.abs(ref.astype(np.float64)).max()
    assert err <= measured_bound * peak, f"{what}: max abs error {err:.3e} > {measured_bound:g} * {peak:.3e}"


@pytest.mark.parametrize("path", ["fp32", "tensor"])
@pytest.mark.parametrize("batch", [1, 24])
def test_mobilenet_v2_cifar(batch, path):
    """MobileNetV2-CIFAR, 10 seeded conv layers at 4 bits, the rest at 8.  The classifier is
    balanced on the 24-image set, so labels spread over the classes, margins are small and the
    tolerance is measured against image-dependent logits instead of a common offset."""
    aiq = binding()
    arch = mobilenet_v2("cifar")
    x24 = gen_images(24, 3, 32, 32, 624)
    params = balance_classifier(arch, gen_model(arch, 2234), x24)
    with compute_path(path):
        model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8))
    scheme = mixed_int4_int8_scheme(53, conv_layer_indices(arch), 10, 43)
    assert (scheme == 4).sum() == 10 and scheme[-1] == 8
    x = x24[:batch]
    got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
    ref = O.forward_scheme(arch, bank, scheme, x)
    if batch == 24:
        assert len(np.unique(O.predict(ref))) >= 5           # the arg-max rule has something to check
    if path == "fp32":
        assert_logits_close(got, ref, f"mbv2 cifar batch={batch}")
    else:
        assert_tensor_path_logits(got, ref, f"mbv2 cifar batch={batch}")
    assert_preds_match(O.predict(got), O.predict(ref), O.top2_margin(ref), "mbv2 cifar")


def test_mobilenet_v2_cifar_batch256_sampled():
    """The batch-256 case of the MobileNetV2-CIFAR workload (the launch shapes of the large
    batch: row-walking depthwise kernel, many-tile pointwise launches) on the tensor path; the
    oracle computes 16 of the 256 images."""
    aiq = binding()
    arch = mobilenet_v2("cifar")
    x = gen_images(256, 3, 32, 32, 856)
    sample = np.arange(5, 256, 16)
    params = balance_classifier(arch, gen_model(arch, 2234), x[sample])
    model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8))
    scheme = mixed_int4_int8_scheme(53, conv_layer_indices(arch), 10, 43)
    got = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
    ref = O.forward_scheme(arch, bank, scheme, x[sample])
    assert len(np.unique(O.predict(ref))) >= 3                # 16 images: several classes, small margins
    assert_tensor_path_logits(got[sample], ref, "mbv2 cifar batch=256")
    assert_preds_match(O.predict(got[sample]), O.predict(ref), O.top2_margin(ref), "mbv2 cifar batch=256")
    # the same images alone give the same logits: no dependence on the batch around them (with the same
    # kernels: the default policy fuses some inverted-residual blocks at batch 256 and none at batch 16)
    alone = model.aiq_forward(scheme, to_dev(x[sample])).cpu().numpy()
    assert_tensor_path_logits(alone, ref, "mbv2 cifar, the sampled images alone")
    aiq.aiq_set_fusion(True, True, inverted_residual=False)
    try:
        got_plain = model.aiq_forward(scheme, to_dev(x)).cpu().numpy()
        alone_plain = model.aiq_forward(scheme, to_dev(x[sample])).cpu().numpy()
    finally:
        aiq.aiq_set_fusion(True, True)
    assert np.array_equal(alone_plain, got_plain[sample])
    assert np.array_equal(alone_plain, alone)


@pytest.mark.parametrize("path", ["fp32", "tensor"])
def test_mobilenet_v2_imagenet_shape(path):
    aiq = binding()
    arch = mobilenet_v2("imagenet")
    params = gen_model(arch, 4234)
    with compute_path(path):
        model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8, 16, 32))
    x = gen_images(3, 3, 224, 224, 4235)
    schemes = coordinate_step_schemes(53, conv_layer_indices(arch))
    for j in (0, 1, 2, 30):
        got = model.aiq_forward(schemes[j], to_dev(x)).cpu().numpy()
        ref = O.forward_scheme(arch, bank, schemes[j], x)
        assert got.shape == (3, 1000)
        if path == "fp32":
            assert_logits_close(got, ref, f"mbv2 imagenet scheme {j}")
        else:
            assert_logits_close_tensor(got, ref, f"mbv2 imagenet scheme {j}")
            assert_preds_match(O.predict(got), O.predict(ref), O.top2_margin(ref), "mbv2 imagenet")


@pytest.mark.parametrize("path", ["fp32", "tensor", "tiles"])
def test_eval_schemes_greedy_step_resnet20(path):
    """One greedy step: 21 candidates, each lowering one conv layer of an all-8 scheme to 4
    bits.  Counts, predictions and accuracies against the oracle; sharing on/off and the
    chunk size must not change a single count."""
    import torch
    aiq = binding()
    arch = resnet20()
    x = gen_images(176, 3, 32, 32, 5679)
    params = balance_classifier(arch, gen_model(arch, 1234), x)
    with compute_path(path):
        model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8))
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    assert len(np.unique(labels)) >= 5                       # the balanced classifier spreads labels
    schemes = one_layer_lowered_schemes(22, conv_layer_indices(arch))
    assert schemes.shape == (21, 22)
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    assert len(set(ocounts.tolist())) > 1                    # the candidates really differ
    xd, ld = to_dev(x), to_dev(labels)
    results = []
    for chunk, share in ((64, True), (64, False), (50, True), (176, True), (7, True)):
        aiq.aiq_set_eval_options(chunk, share)
        preds = torch.full((21, 176), -1, dtype=torch.int32, device="cuda")
        acc, counts = model.aiq_eval_schemes(schemes, xd, ld, preds=preds, chunk=chunk)
        stats = aiq.aiq_last_call_stats()
        results.append((counts.copy(), preds.cpu().numpy(), stats))
        assert np.allclose(acc, counts / 176.0)
    aiq.aiq_set_eval_options(0, True)
    counts0, preds0, stats0 = results[0]
    for counts, preds, _ in results[1:]:
        assert np.array_equal(counts, counts0)
        assert np.array_equal(preds, preds0)
    assert_preds_match(preds0, opreds, omargins, "greedy step")
    slack = (omargins <= 1e-2).sum(axis=1)
    assert np.all(np.abs(counts0 - ocounts) <= slack)
    assert np.array_equal((preds0 == labels[None, :]).sum(axis=1), counts0)
    # prefix sharing does strictly less work than 21 independent passes
    assert stats0["layer_evals"] < results[1][2]["layer_evals"] == stats0["layer_evals_unshared"]
    assert stats0["kernel_launches"] > 0


def test_eval_schemes_duplicates_fc_candidates_and_tiny_net():
    import torch
    aiq = binding()
    arch = tiny_net()
    x = gen_images(45, 3, 8, 8, 71)
    params = balance_classifier(arch, gen_model(arch, 99), x)
    model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params)
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    L = model.n_layers
    schemes = np.concatenate([
        one_layer_lowered_schemes(L, list(range(L))),                 # includes the classifier
        coordinate_step_schemes(L, list(range(L))),
        np.stack([gen_random_scheme(L, s) for s in range(5)]),
        np.full((2, L), 32, np.uint8),                                # duplicates
        one_layer_lowered_schemes(L, [3]),                            # duplicate of row 3
    ])
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    preds = torch.full((len(schemes), 45), -1, dtype=torch.int32, device="cuda")
    aiq.aiq_set_eval_options(16, True)
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=16)
    aiq.aiq_set_eval_options(0, True)
    p = preds.cpu().numpy()
    assert_preds_match(p, opreds, omargins, "tiny eval")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    assert np.array_equal(p[-1], p[3]) and np.array_equal(p[-2], p[-3])
    assert counts[-2] == counts[-3] == 45                             # all-32 scheme agrees with itself
    assert acc[-2] == 1.0


def test_eval_schemes_coordinate_step_mobilenet_v2_imagenet():
    """The coordinate-descent step on ImageNet-shaped MobileNetV2 at reduced size: candidates
    that move one conv layer of an all-8 scheme to 32, 16 or 4 bits (so float32-kernel layers
    sit inside a tensor-path model), evaluated with shared prefixes and a ragged last chunk.
    Counts and predictions against the oracle; the chunk size must not change a count."""
    import torch
    aiq = binding()
    arch = mobilenet_v2("imagenet")
    x = gen_images(5, 3, 224, 224, 4236)
    params = balance_classifier(arch, gen_model(arch, 4234), x)
    model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8, 16, 32))
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    all_schemes = coordinate_step_schemes(53, conv_layer_indices(arch))
    assert all_schemes.shape == (52, 53)
    schemes = all_schemes[[0, 1, 2, 10, 20, 31, 40, 47, 51]]
    assert {int(b) for b in np.unique(schemes)} == {4, 8, 16, 32}
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    xd, ld = to_dev(x), to_dev(labels)
    got = []
    for chunk in (2, 5):
        aiq.aiq_set_eval_options(chunk, True)
        preds = torch.full((len(schemes), 5), -1, dtype=torch.int32, device="cuda")
        acc, counts = model.aiq_eval_schemes(schemes, xd, ld, preds=preds, chunk=chunk)
        got.append((counts.copy(), preds.cpu().numpy()))
        assert np.allclose(acc, counts / 5.0)
    aiq.aiq_set_eval_options(0, True)
    assert np.array_equal(got[0][0], got[1][0]) and np.array_equal(got[0][1], got[1][1])
    counts, p = got[0]
    assert_preds_match(p, opreds, omargins, "coordinate step")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    assert np.array_equal((p == labels[None, :]).sum(axis=1), counts)
    ai = [model.aiq_scheme_ai(sc)[0] for sc in schemes]
    oai = [O.scheme_ai(arch, sc)[0] for sc in schemes]
    assert np.allclose(ai, oai, rtol=1e-12)


def test_coordinate_step_all_52_candidates_mobilenet_v2_imagenet():
    """The benchmark's second sweep workload at reduced image count: all 52 candidates of the
    coordinate-descent slice on 3 images against the oracle, and the base (all-8) scheme on 24
    images in the benchmark's pass size with 6 of them checked by the oracle."""
    import torch
    from bench import eval_workload
    aiq = binding()
    wl = eval_workload("mbv2_imagenet_cd_step")
    arch, schemes = wl["arch"], wl["schemes"]
    assert schemes.shape == (52, 53)
    x = gen_images(24, 3, 224, 224, 4240)
    sample = np.arange(0, 24, 4)
    params = balance_classifier(arch, gen_model(arch, wl["seed_model"]), x[sample])
    model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8, 16, 32))
    labels = np.zeros(24, np.int32)
    labels[sample] = O.predict(O.forward_fp32_unquantized(arch, folded, x[sample]))
    # (a) every candidate on three images
    sub = sample[:3]
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x[sub], labels[sub])
    preds = torch.full((52, 3), -1, dtype=torch.int32, device="cuda")
    aiq.aiq_set_eval_options(wl["chunk"], True)
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x[sub]), to_dev(labels[sub]), preds=preds, chunk=wl["chunk"])
    p = preds.cpu().numpy()
    assert_preds_match(p, opreds, omargins, "coordinate step, all candidates")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    # (b) the base scheme over the larger set, sampled
    base = np.full((1, 53), 8, np.uint8)
    preds = torch.full((1, 24), -1, dtype=torch.int32, device="cuda")
    acc, counts = model.aiq_eval_schemes(base, to_dev(x), to_dev(labels), preds=preds, chunk=wl["chunk"])
    aiq.aiq_set_eval_options(0, True)
    p = preds.cpu().numpy()
    assert np.array_equal((p == labels[None, :]).sum(axis=1), counts)
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, base, x[sample], labels[sample])
    assert_preds_match(p[:, sample], opreds, omargins, "coordinate step, base scheme")
    model.close()


@pytest.mark.parametrize("path", ["fp32", "tensor", "tiles"])
@pytest.mark.parametrize("make", [heavy_early_resnet20, plain_convnet20])
def test_structural_variants_of_section_4_5(make, path):
    """HeavyEarlyResNet20 (wide layers first, width changes at stride 1, 64 -> 32 -> 16 channels)
    and PlainConvNet20 (20 plain 64-channel convolutions): forward logits of mixed schemes and a
    greedy step over every conv layer against the oracle."""
    import torch
    aiq = binding()
    arch = make()
    L = len(arch["layers"])
    x = gen_images(40, 3, 32, 32, 4501)
    params = balance_classifier(arch, gen_model(arch, 4500), x)
    with compute_path(path):
        model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8, 16, 32))
    for seed in (1, 2):
        scheme = gen_random_scheme(L, seed)
        got = model.aiq_forward(scheme, to_dev(x[:9])).cpu().numpy()
        ref = O.forward_scheme(arch, bank, scheme, x[:9])
        if path == "fp32":
            assert_logits_close(got, ref, f"{arch['name']} scheme seed {seed}")
        else:
            assert_logits_close_tensor(got, ref, f"{arch['name']} scheme seed {seed}")
            assert_preds_match(O.predict(got), O.predict(ref), O.top2_margin(ref), arch["name"])
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    schemes = one_layer_lowered_schemes(L, conv_layer_indices(arch))
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x, labels)
    preds = torch.full((len(schemes), 40), -1, dtype=torch.int32, device="cuda")
    aiq.aiq_set_eval_options(16, True)
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=16)
    aiq.aiq_set_eval_options(0, True)
    p = preds.cpu().numpy()
    assert_preds_match(p, opreds, omargins, arch["name"] + " greedy step")
    assert np.all(np.abs(counts - ocounts) <= (omargins <= 1e-2).sum(axis=1))
    assert abs(model.aiq_scheme_ai(schemes[3])[0] - O.scheme_ai(arch, schemes[3])[0]) < 1e-9


def test_forward_and_eval_errors():
    import torch
    aiq = binding()
    arch = tiny_net()
    model = aiq.Model(arch, gen_model(arch, 1))
    x = to_dev(gen_images(4, 3, 8, 8, 2))
    bad = np.full(model.n_layers, 8, np.uint8)
    bad[2] = 7
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_forward(bad, x)
    assert e.value.status == aiq.ERR_UNSUPPORTED_BITS
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_forward(np.full(model.n_layers, 8, np.uint8), x, workspace=small)
    assert e.value.status == aiq.ERR_WORKSPACE_TOO_SMALL
    labels = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_eval_schemes(bad[None, :], x, labels)
    assert e.value.status == aiq.ERR_UNSUPPORTED_BITS
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_eval_schemes(np.full((1, model.n_layers), 8, np.uint8), x, labels, workspace=small)
    assert e.value.status == aiq.ERR_WORKSPACE_TOO_SMALL


def test_full_size_greedy_step_sampled_against_oracle():
    """The benchmark's configuration: 10,000 images, 21 candidate schemes, the benchmark's pass
    size, tensor-core path.  The oracle cannot run 210,000 forwards, so predictions are compared on
    a sample of images it computes one by one; over the whole set the counts must equal the
    number of predictions that match the labels."""
    import torch
    aiq = binding()
    arch = resnet20()
    n = 10000
    x = gen_images(n, 3, 32, 32, 5679)
    sample = np.arange(0, n, 131)[:72]                      # 72 images spread over all chunks
    params = balance_classifier(arch, gen_model(arch, 1234), x[sample])
    model = aiq.Model(arch, params)
    folded, bank = _oracle_bank(arch, params, (4, 8))
    schemes = one_layer_lowered_schemes(22, conv_layer_indices(arch))
    labels = np.random.default_rng(3).integers(0, 10, n).astype(np.int32)
    labels[sample] = O.predict(O.forward_fp32_unquantized(arch, folded, x[sample]))
    oacc, ocounts, opreds, omargins = O.eval_schemes(arch, bank, schemes, x[sample], labels[sample])
    preds = torch.full((21, n), -1, dtype=torch.int32, device="cuda")
    from bench import DEFAULT_CHUNK
    aiq.aiq_set_eval_options(DEFAULT_CHUNK, True)
    acc, counts = model.aiq_eval_schemes(schemes, to_dev(x), to_dev(labels), preds=preds, chunk=DEFAULT_CHUNK)
    aiq.aiq_set_eval_options(0, True)
    p = preds.cpu().numpy()
    assert p.min() >= 0 and p.max() <= 9
    assert np.array_equal((p == labels[None, :]).sum(axis=1), counts)
    assert np.allclose(acc, counts / float(n))
    assert_preds_match(p[:, sample], opreds, omargins, "full size sample")
    assert len(np.unique(p[0])) >= 5

"""Greedy search and coordinate descent (Section 2.2) of the CUDA library against the oracle."""
import numpy as np
import pytest

from aiq_workloads import resnet20, tiny_net, gen_model, gen_images
from oracle import aiq_oracle as O
from gpu_util import binding, to_dev

pytestmark = pytest.mark.gpu


def _setup(arch, seed_model, x, balanced):
    """Model, oracle bank and labels.  `balanced`: shift the classifier bias by the oracle's mean
    logits so that labels spread over the classes and margins are small (accuracy then moves
    with every quantization step); otherwise the random-init network puts nearly all images
    in one class with wide margins, and the searches are decided by AI alone."""
    params = gen_model(arch, seed_model)
    folded = O.fold_model(arch, params)
    if balanced:
        mean_logits = O.forward_fp32_unquantized(arch, folded, x).astype(np.float64).mean(axis=0)
        params = [dict(p) for p in params]
        params[-1]["bias"] = (params[-1]["bias"].astype(np.float64) - mean_logits).astype(np.float32)
        folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded, (4, 8, 32))
    labels = O.predict(O.forward_fp32_unquantized(arch, folded, x))
    return params, bank, labels


def _oracle_fns(arch, bank, x, labels):
    slack = {}

    def acc_fn(schemes):
        acc, counts, preds, margins = O.eval_schemes(arch, bank, schemes, x, labels)
        for s, m in zip(schemes, margins):
            slack[bytes(s)] = int((m <= 1e-2).sum())
        return acc

    def ai_fn(s):
        return O.scheme_ai(arch, s)[0]

    return acc_fn, ai_fn, slack


def _check_trace(kind, got_scheme, got_steps, ref_scheme, ref_trace, slack, n_images, lam):
    """Equal trajectories when no image of any evaluated scheme sits inside the arg-max
    margin (then the counts agree exactly); otherwise the losses may differ by what those
    images can move, and the final schemes must still be explained by it."""
    undecided = sum(slack.values())
    ref = [(t[0], t[1], t[2]) for t in ref_trace]
    got = [(t["layer"], t["bits"], t["accepted"]) for t in got_steps]
    if undecided == 0:
        assert got == ref, f"{kind}: {got} vs {ref}"
        assert got_scheme.tolist() == ref_scheme.tolist()
        for g, r in zip(got_steps, ref_trace):
            assert abs(g["loss"] - r[3]) <= 1e-9 * max(1.0, abs(r[3]))
    else:
        eps = (1.0 - lam) * 100.0 * max(slack.values()) / n_images
        n = min(len(got_steps), len(ref_trace))
        for g, r in zip(got_steps[:n], ref_trace[:n]):
            if (g["layer"], g["bits"], g["accepted"]) != (r[0], r[1], r[2]):
                break                                   # a near-tie went the other way: stop comparing
            assert abs(g["loss"] - r[3]) <= 2 * eps + 1e-9


@pytest.mark.parametrize("balanced", [False, True])
@pytest.mark.parametrize("lam", [0.9, 0.02])
def test_searches_on_tiny_net_match_the_oracle(lam, balanced):
    aiq = binding()
    arch = tiny_net()
    x = gen_images(45, 3, 8, 8, 71)
    params, bank, labels = _setup(arch, 99, x, balanced)
    model = aiq.Model(arch, params)
    L = model.n_layers
    xd, ld = to_dev(x), to_dev(labels)

    acc_fn, ai_fn, slack = _oracle_fns(arch, bank, x, labels)
    ref_q, ref_t = O.greedy_search(L, acc_fn, ai_fn, lam, options=(8, 4))
    got_q, got_t = model.aiq_search_greedy(xd, ld, lam, options=(8, 4), chunk=16)
    _check_trace("greedy", got_q, got_t, ref_q, ref_t, slack, 45, lam)
    assert all(b in (32, 8, 4) for b in got_q)
    ai = model.aiq_scheme_ai(got_q)[0]
    if got_t and got_t[-1]["accepted"]:
        assert abs(got_t[-1]["ai"] - ai) < 1e-9

    acc_fn, ai_fn, slack = _oracle_fns(arch, bank, x, labels)
    ref_q, ref_t = O.coordinate_descent(L, acc_fn, ai_fn, lam, options=(32, 8, 4), max_passes=4)
    got_q, got_t = model.aiq_search_coordinate_descent(xd, ld, lam, options=(32, 8, 4), max_passes=4, chunk=16)
    _check_trace("coordinate descent", got_q, got_t, ref_q, ref_t, slack, 45, lam)


@pytest.mark.parametrize("balanced", [False, True])
def test_greedy_on_resnet20_layer_subset_matches_the_oracle(balanced):
    """ResNet-20, moves restricted to four layers so that the oracle can follow: a stage-2
    convolution, two stage-3 convolutions and the classifier."""
    aiq = binding()
    arch = resnet20()
    x = gen_images(48, 3, 32, 32, 5680)
    params, bank, labels = _setup(arch, 1234, x, balanced)
    model = aiq.Model(arch, params)
    layers = [13, 18, 19, 21]
    acc_fn, ai_fn, slack = _oracle_fns(arch, bank, x, labels)
    ref_q, ref_t = O.greedy_search(22, acc_fn, ai_fn, 0.9, options=(8, 4), layers=layers)
    got_q, got_t = model.aiq_search_greedy(to_dev(x), to_dev(labels), 0.9, options=(8, 4), layers=layers, chunk=48)
    _check_trace("greedy resnet20", got_q, got_t, ref_q, ref_t, slack, 48, 0.9)
    assert [int(got_q[i]) for i in range(22) if i not in layers] == [32] * 18
    assert got_t[0]["candidates"] == 8


def test_search_argument_errors():
    import torch
    aiq = binding()
    arch = tiny_net()
    model = aiq.Model(arch, gen_model(arch, 1))
    x = to_dev(gen_images(4, 3, 8, 8, 2))
    labels = torch.zeros(4, dtype=torch.int32, device="cuda")
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_search_greedy(x, labels, 1.5)
    assert e.value.status == aiq.ERR_INVALID_ARG
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_search_greedy(x, labels, 0.9, options=(8, 5))
    assert e.value.status == aiq.ERR_UNSUPPORTED_BITS
    with pytest.raises(aiq.AiqError) as e:
        model.aiq_search_coordinate_descent(x, labels, 0.9, layers=[0, 99])
    assert e.value.status == aiq.ERR_INVALID_ARG

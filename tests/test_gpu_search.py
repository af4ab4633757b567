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


class _Evaluations:
    """acc_fn / ai_fn pair for the oracle's search drivers.

    `source` = "oracle": accuracies come from the oracle's own forward passes.
    `source` = "gpu": accuracies are count / n of the library's aiq_eval_schemes on the same
    schemes, so the oracle's search logic (candidate set, arg-min, tie-breaking, accept rule,
    loss) runs on exactly the numbers the library's search sees.  Either way the oracle's
    counts and arg-max margins of every evaluated scheme are recorded for the count check."""

    def __init__(self, arch, bank, x, labels, source, model=None, xd=None, ld=None, chunk=16):
        self.arch, self.bank, self.x, self.labels, self.source = arch, bank, x, labels, source
        self.model, self.xd, self.ld, self.chunk = model, xd, ld, chunk
        self.oracle_counts, self.slack, self.gpu_counts = {}, {}, {}

    def acc_fn(self, schemes):
        schemes = np.ascontiguousarray(schemes, dtype=np.uint8)
        acc, counts, _preds, margins = O.eval_schemes(self.arch, self.bank, schemes, self.x, self.labels)
        for s, c, m in zip(schemes, counts, margins):
            self.oracle_counts[bytes(s)] = int(c)
            self.slack[bytes(s)] = int((m <= 1e-2).sum())
        if self.source == "oracle":
            return acc
        _gacc, gcounts = self.model.aiq_eval_schemes(schemes, self.xd, self.ld, chunk=self.chunk)
        for s, c in zip(schemes, gcounts):
            self.gpu_counts[bytes(s)] = int(c)
        return gcounts.astype(np.float64) / float(len(self.labels))

    def ai_fn(self, s):
        return O.scheme_ai(self.arch, s)[0]


def _check_search(kind, got_scheme, got_steps, ev, run_oracle_search):
    """Two checks that hold whatever the arg-max margins are.

    (1) The oracle's search driver, fed with the library's own counts, must reproduce the
        library's trajectory move by move (layer, bit-width, accept flag), its losses to 1e-9
        and its final scheme: this pins the search logic of the library.
    (2) For every scheme that search evaluated, the library's count may differ from the
        oracle's by at most the number of images whose oracle margin is within 1e-2: this
        pins the numbers the search logic was fed with.
    Where no evaluated image sits inside the margin the two together mean: same trajectory
    as the pure oracle search, which is then asserted as well."""
    ref_scheme, ref_trace = run_oracle_search(ev.acc_fn, ev.ai_fn)
    ref = [(t[0], t[1], t[2]) for t in ref_trace]
    got = [(t["layer"], t["bits"], t["accepted"]) for t in got_steps]
    assert got == ref, f"{kind}: {got} vs {ref}"
    assert got_scheme.tolist() == ref_scheme.tolist(), kind
    for g, r in zip(got_steps, ref_trace):
        assert abs(g["loss"] - r[3]) <= 1e-9 * max(1.0, abs(r[3])), kind
    assert ev.gpu_counts, kind
    for key, c in ev.gpu_counts.items():
        assert abs(c - ev.oracle_counts[key]) <= ev.slack[key], (kind, list(key), c, ev.oracle_counts[key])
    return sum(ev.slack.values())


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

    got_q, got_t = model.aiq_search_greedy(xd, ld, lam, options=(8, 4), chunk=16)
    ev = _Evaluations(arch, bank, x, labels, "gpu", model, xd, ld)
    undecided = _check_search("greedy", got_q, got_t, ev,
                              lambda a, f: O.greedy_search(L, a, f, lam, options=(8, 4)))
    if undecided == 0:                                # then the pure oracle search must agree too
        ev0 = _Evaluations(arch, bank, x, labels, "oracle")
        ref_q, _ = O.greedy_search(L, ev0.acc_fn, ev0.ai_fn, lam, options=(8, 4))
        assert got_q.tolist() == ref_q.tolist()
    assert all(b in (32, 8, 4) for b in got_q)
    ai = model.aiq_scheme_ai(got_q)[0]
    if got_t and got_t[-1]["accepted"]:
        assert abs(got_t[-1]["ai"] - ai) < 1e-9

    got_q, got_t = model.aiq_search_coordinate_descent(xd, ld, lam, options=(32, 8, 4), max_passes=4, chunk=16)
    ev = _Evaluations(arch, bank, x, labels, "gpu", model, xd, ld)
    _check_search("coordinate descent", got_q, got_t, ev,
                  lambda a, f: O.coordinate_descent(L, a, f, lam, options=(32, 8, 4), max_passes=4))
    if balanced:
        # accuracy really takes part: the evaluated schemes do not all have the same count
        assert len(set(ev.gpu_counts.values())) > 1


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
    xd, ld = to_dev(x), to_dev(labels)
    got_q, got_t = model.aiq_search_greedy(xd, ld, 0.9, options=(8, 4), layers=layers, chunk=48)
    ev = _Evaluations(arch, bank, x, labels, "gpu", model, xd, ld, chunk=48)
    undecided = _check_search("greedy resnet20", got_q, got_t, ev,
                              lambda a, f: O.greedy_search(22, a, f, 0.9, options=(8, 4), layers=layers))
    if undecided == 0:
        ev0 = _Evaluations(arch, bank, x, labels, "oracle")
        ref_q, ref_t = O.greedy_search(22, ev0.acc_fn, ev0.ai_fn, 0.9, options=(8, 4), layers=layers)
        assert got_q.tolist() == ref_q.tolist()
        assert [(t["layer"], t["bits"], t["accepted"]) for t in got_t] == [(t[0], t[1], t[2]) for t in ref_t]
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

"""Seeded random tensors for the workloads (NumPy PCG64, fixed draw order).

Everything returned is a plain NumPy array (or a list of dicts of arrays) that
is handed unchanged to whichever implementation consumes it.  No arithmetic of
the method lives here: a model is its *unfolded* FP32 weights and batch-norm
vectors, exactly what a trained checkpoint would hold.
"""
import numpy as np

BIT_CHOICES = (32, 16, 8, 4)


def gen_model(arch, seed):
    """Random-init parameters for every layer of `arch`, in layer order.

    Per conv / depthwise layer, drawn in this order from one generator:
      W      ~ N(0, 2/fan_in), fan_in = (cin/groups)*k*k, shape [cout][cin/groups][k][k]
      gamma  ~ U(0.5, 1.5), beta ~ N(0, 0.1), mean ~ N(0, 0.1), var ~ U(0.5, 1.5), each [cout]
    Per fc layer: W ~ N(0, 2/cin) of shape [cout][cin], bias ~ N(0, 0.1) of shape [cout].
    All float32.
    """
    rng = np.random.default_rng(seed)
    params = []
    for layer in arch["layers"]:
        cout, cin, k = layer["cout"], layer["cin"], layer["k"]
        if layer["kind"] == "fc":
            w = (rng.standard_normal((cout, cin), dtype=np.float32)
                 * np.float32(np.sqrt(2.0 / cin)))
            bias = rng.standard_normal(cout, dtype=np.float32) * np.float32(0.1)
            params.append(dict(W=w, bias=bias))
            continue
        cin_g = 1 if layer["kind"] == "dw" else cin
        fan_in = cin_g * k * k
        w = (rng.standard_normal((cout, cin_g, k, k), dtype=np.float32)
             * np.float32(np.sqrt(2.0 / fan_in)))
        gamma = rng.uniform(0.5, 1.5, cout).astype(np.float32)
        beta = rng.standard_normal(cout, dtype=np.float32) * np.float32(0.1)
        mean = rng.standard_normal(cout, dtype=np.float32) * np.float32(0.1)
        var = rng.uniform(0.5, 1.5, cout).astype(np.float32)
        params.append(dict(W=w, gamma=gamma, beta=beta, mean=mean, var=var))
    return params


def gen_images(n, c, h, w, seed):
    """`n` images, float32 NCHW, every value ~ N(0, 1)."""
    rng = np.random.default_rng(seed)
    return rng.standard_normal((n, c, h, w), dtype=np.float32)


def gen_random_scheme(n_layers, seed):
    """One bit-width per layer, uniform over {32, 16, 8, 4}."""
    rng = np.random.default_rng(seed)
    return np.asarray(BIT_CHOICES, dtype=np.uint8)[rng.integers(0, 4, n_layers)]


def one_layer_lowered_schemes(n_layers, candidates, base=8, low=4):
    """One greedy step: scheme j = all-`base` with layer candidates[j] set to `low`."""
    s = np.full((len(candidates), n_layers), base, dtype=np.uint8)
    for j, i in enumerate(candidates):
        s[j, i] = low
    return s


def coordinate_step_schemes(n_layers, candidates, base=8, alternatives=(32, 16, 4)):
    """One coordinate-descent sweep slice: scheme j changes layer candidates[j] only,
    to alternatives[j mod len(alternatives)]."""
    s = np.full((len(candidates), n_layers), base, dtype=np.uint8)
    for j, i in enumerate(candidates):
        s[j, i] = alternatives[j % len(alternatives)]
    return s


def mixed_int4_int8_scheme(n_layers, candidates, n_low, seed):
    """`n_low` of `candidates` (chosen without replacement) at 4 bits, the rest at 8."""
    rng = np.random.default_rng(seed)
    pick = rng.choice(np.asarray(candidates), size=n_low, replace=False)
    s = np.full(n_layers, 8, dtype=np.uint8)
    s[pick] = 4
    return s


def gen_linear_case(n, k, m, seed, w_std=0.02):
    """Standalone linear layer: W [n][k] ~ N(0, w_std^2), x [m][k] ~ N(0, 1), float32."""
    rng = np.random.default_rng(seed)
    w = rng.standard_normal((n, k), dtype=np.float32) * np.float32(w_std)
    x = rng.standard_normal((m, k), dtype=np.float32)
    return w, x

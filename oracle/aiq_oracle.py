"""CPU oracle for AIQ scheme evaluation (test infrastructure, not a product path).

A plain, slow NumPy statement of what the hot path computes: batch-norm folding,
the per-layer weight quantizer, the quantized CNN forward pass, top-1 agreement,
the analytic global arithmetic intensity, and the two searches of Section 2.2 over the
AIQ objective (the units inside the objective are a stated reading: parity unpinned).  Only tests, the smoke check and
the benchmark's CPU-baseline leg may import this module; the CUDA library shares
no code with it.

Where the paper fixes the definition the function cites it.  The paper names the
bit-width set and the objective but gives neither a quantizer formula nor an AI
formula; the readings used are stated in each docstring.

Precision: folding and quantization are float32 with every operation rounded
once (NumPy float32 ufuncs are IEEE, unfused).  The forward pass accumulates
every output element in float64 and rounds once to float32 per materialised
tensor.
"""
import numpy as np

EPS_BN = np.float32(1e-5)
ALLOWED_BITS = (4, 8, 16, 32)


# ----------------------------------------------------------------------------
# Batch-norm folding
# ----------------------------------------------------------------------------
def fold_bn(W, gamma, beta, mean, var, eps=EPS_BN):
    """Fold inference batch-norm into the preceding convolution.

    The paper evaluates a trained PyTorch model (Section 3) and does not mention
    folding; folding before quantizing is this implementation's stated reading.
    g = gamma / sqrt(var + eps);  W' = W * g (per output channel);  b' = beta - mean * g.
    float32, each operation rounded once.
    """
    W = np.asarray(W, dtype=np.float32)
    g = gamma.astype(np.float32) / np.sqrt(var.astype(np.float32) + np.float32(eps))
    Wf = W * g.reshape((-1,) + (1,) * (W.ndim - 1))
    bf = beta.astype(np.float32) - mean.astype(np.float32) * g
    return Wf.astype(np.float32), bf.astype(np.float32)


def fold_model(arch, params):
    """Folded (W' [cout][K], b' [cout]) for every layer; fc layers pass through."""
    out = []
    for layer, p in zip(arch["layers"], params):
        if layer["has_bn"]:
            Wf, bf = fold_bn(p["W"], p["gamma"], p["beta"], p["mean"], p["var"])
        else:
            Wf, bf = p["W"].astype(np.float32), p["bias"].astype(np.float32)
        out.append((Wf.reshape(Wf.shape[0], -1), bf))
    return out


# ----------------------------------------------------------------------------
# Quantizer (Section 2.1: q_i in Q; Q = {FP32, INT8, INT4}, plus a 16-bit level)
# ----------------------------------------------------------------------------
def quantize_rows(W, bits, per_tensor=False):
    """Quantize a folded weight matrix W [N][K] (one row per output channel).

    Section 2.1 assigns each layer a bit-width but prints no formula.  Reading:
    symmetric, per output channel, max-abs scale, round half to even.
      bits 4 / 8:  qmax = 2^(bits-1) - 1;  amax_n = max_k |W[n,k]|;
                   s_n = amax_n / qmax (float32 division), s_n = 1 if amax_n == 0;
                   code = clamp(rint(W[n,k] / s_n), -2^(bits-1), 2^(bits-1) - 1)
      bits 16:     IEEE half, round to nearest even; s_n = 1
      bits 32:     unchanged; s_n = 1
    per_tensor=True is the variant with one scale for the whole tensor (the paper lists
    per-channel effects as future work in Section 6, so its own experiments most likely used
    this granularity): amax = max over all of W, every entry of `scales` holds amax / qmax.
    Returns (values, scales): values is int8 codes, float16 or float32; scales float32 [N].
    Non-finite weights raise ValueError.
    """
    if bits not in ALLOWED_BITS:
        raise ValueError(f"unsupported bit-width {bits}")
    W = np.ascontiguousarray(W, dtype=np.float32)
    if W.ndim != 2:
        raise ValueError("W must be [N][K]")
    if not np.all(np.isfinite(W)):
        raise ValueError("non-finite weight")
    n = W.shape[0]
    ones = np.ones(n, dtype=np.float32)
    if bits == 32:
        return W.copy(), ones
    if bits == 16:
        return W.astype(np.float16), ones
    qmax = np.float32(2 ** (bits - 1) - 1)
    amax = np.max(np.abs(W), axis=1) if W.shape[1] else np.zeros(n, np.float32)
    if per_tensor:
        amax = np.full(n, np.max(amax) if n else 0.0, dtype=np.float32)
    s = (amax / qmax).astype(np.float32)
    s[amax == 0] = np.float32(1.0)
    q = np.rint(W / s[:, None])
    q = np.clip(q, -(2 ** (bits - 1)), 2 ** (bits - 1) - 1)
    return q.astype(np.int8), s


def dequantize_rows(values, scales, bits):
    """w_hat = float32(code) * s_n (one float32 multiply) at 4/8 bits; float32(half) at 16;
    the weight itself at 32."""
    if bits in (4, 8):
        return values.astype(np.float32) * scales[:, None].astype(np.float32)
    return values.astype(np.float32)


def padded_k(K):
    """Row length in elements of the packed store: K rounded up to a multiple of 32."""
    return (K + 31) // 32 * 32


def packed_row_bytes(K, bits):
    return padded_k(K) * bits // 8


def pack_rows(values, bits):
    """Packed byte image of quantized rows: row-major, rows padded with zero elements to
    padded_k(K).  4 bits: byte j holds element 2j in its low nibble and element 2j+1 in
    its high nibble (two's complement).  8 bits: int8.  16: IEEE half, little endian.
    32: float32, little endian."""
    n, K = values.shape
    kp = padded_k(K)
    if bits == 4:
        c = np.zeros((n, kp), dtype=np.uint8)
        c[:, :K] = values.astype(np.int8).view(np.uint8) & 0xF
        return (c[:, 0::2] | (c[:, 1::2] << 4)).astype(np.uint8)
    dt = {8: np.int8, 16: np.float16, 32: np.float32}[bits]
    c = np.zeros((n, kp), dtype=dt)
    c[:, :K] = values.astype(dt)
    return c.view(np.uint8).reshape(n, -1)


def unpack_rows(packed, K, bits):
    """Inverse of pack_rows: the logical elements [N][K]."""
    n = packed.shape[0]
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    if bits == 4:
        lo = (packed & 0xF).astype(np.int16)
        hi = (packed >> 4).astype(np.int16)
        c = np.empty((n, packed.shape[1] * 2), dtype=np.int16)
        c[:, 0::2] = lo
        c[:, 1::2] = hi
        c = np.where(c >= 8, c - 16, c)
        return c[:, :K].astype(np.int8)
    dt = {8: np.int8, 16: np.float16, 32: np.float32}[bits]
    return packed.view(dt).reshape(n, -1)[:, :K].copy()


# ----------------------------------------------------------------------------
# Forward pass (Section 1: "measure the model's accuracy empirically")
# ----------------------------------------------------------------------------
def _activate(y, act):
    if act == "relu":
        return np.maximum(y, 0.0)
    if act == "relu6":
        return np.minimum(np.maximum(y, 0.0), 6.0)
    if act == "none":
        return y
    raise ValueError(act)


def out_hw(h, k, stride, pad):
    return (h + 2 * pad - k) // stride + 1


def conv2d_f64(x, w, stride, pad, depthwise=False):
    """Cross-correlation of x [B][C][H][W] with w [Cout][C or 1][k][k], zero padding,
    float64 accumulation.  y[b,n,oy,ox] = sum_{c,r,t} w[n,c,r,t] * x[b,c,oy*s+r-p,ox*s+t-p].
    The sum over taps (r, t) is an explicit loop; the sum over channels of one tap is a
    float64 matmul (dense) or an elementwise product (depthwise).
    """
    B, C, H, Wd = x.shape
    cout, _, k, _ = w.shape
    Ho, Wo = out_hw(H, k, stride, pad), out_hw(Wd, k, stride, pad)
    xp = np.zeros((B, C, H + 2 * pad, Wd + 2 * pad), dtype=np.float64)
    xp[:, :, pad:pad + H, pad:pad + Wd] = x
    w64 = w.astype(np.float64)
    y = np.zeros((B, cout, Ho, Wo), dtype=np.float64)
    for r in range(k):
        for t in range(k):
            win = xp[:, :, r:r + (Ho - 1) * stride + 1:stride, t:t + (Wo - 1) * stride + 1:stride]
            if depthwise:
                y += win * w64[None, :, 0, r, t, None, None]
            else:
                # [B][Ho][Wo][C] @ [C][Cout] -> [B][Ho][Wo][Cout]
                y += np.matmul(win.transpose(0, 2, 3, 1), w64[:, :, r, t].T).transpose(0, 3, 1, 2)
    return y


def execution_order(arch):
    """Layer indices in an order where every layer follows its input and its residual
    source (a block's projection is listed after the conv that adds it)."""
    order, done = [], set()

    def visit(i):
        if i < 0 or i in done:
            return
        visit(arch["layers"][i]["input"])
        visit(arch["layers"][i]["residual"])
        done.add(i)
        order.append(i)

    for i in range(len(arch["layers"])):
        visit(i)
    return order


def forward(arch, deq_layers, x):
    """Logits of the network for images x [B][C][H][W] (float32).

    deq_layers[i] = (w_hat float32 [cout][K], b float32 [cout]) - the dequantized folded
    weights.  Every layer output is float64-accumulated, then bias, then residual, then
    activation, then rounded once to float32.  An fc layer takes the float64 mean over
    H x W of its input (rounded to float32) and returns float32 logits.
    Basic block: relu(conv2(relu(conv1(x))) + shortcut(x)); inverted residual:
    project(dw(expand(x))) + x when shapes allow.
    """
    x = np.asarray(x, dtype=np.float32)
    outs = [None] * len(arch["layers"])
    for i in execution_order(arch):
        layer, (w_hat, b) = arch["layers"][i], deq_layers[i]
        src = x if layer["input"] < 0 else outs[layer["input"]]
        if layer["kind"] == "fc":
            pooled = src.astype(np.float64).mean(axis=(2, 3)).astype(np.float32)
            y = np.matmul(pooled.astype(np.float64), w_hat.astype(np.float64).T) + b.astype(np.float64)
            outs[i] = y.astype(np.float32)
            continue
        dw = layer["kind"] == "dw"
        cin_g = 1 if dw else layer["cin"]
        w4 = w_hat.reshape(layer["cout"], cin_g, layer["k"], layer["k"])
        y = conv2d_f64(src, w4, layer["stride"], layer["pad"], depthwise=dw)
        y += b.astype(np.float64)[None, :, None, None]
        if layer["residual"] >= 0:
            y += outs[layer["residual"]].astype(np.float64)
        outs[i] = _activate(y, layer["act"]).astype(np.float32)
    return outs[-1]


def build_weight_bank(folded, bits_set=ALLOWED_BITS, per_tensor=False):
    """bank[i][bits] = (w_hat, b): a layer's quantized weights depend only on (layer, bits)."""
    bank = []
    for Wf, bf in folded:
        entry = {}
        for bits in bits_set:
            v, s = quantize_rows(Wf, bits, per_tensor)
            entry[bits] = (dequantize_rows(v, s, bits), bf)
        bank.append(entry)
    return bank


def forward_scheme(arch, bank, scheme, x, chunk=256):
    """Logits under the scheme q = (q_1 .. q_L) of Section 2.1, in chunks of images."""
    deq = [bank[i][int(b)] for i, b in enumerate(scheme)]
    return np.concatenate([forward(arch, deq, x[i:i + chunk]) for i in range(0, len(x), chunk)])


def forward_fp32_unquantized(arch, folded, x, chunk=256):
    """The folded FP32 model with no quantizer in the path (start point of both searches)."""
    return np.concatenate([forward(arch, folded, x[i:i + chunk]) for i in range(0, len(x), chunk)])


# ----------------------------------------------------------------------------
# Accuracy (Section 2.1: AccLoss(q) is measured, not modelled)
# ----------------------------------------------------------------------------
def predict(logits):
    """Lowest index attaining the maximum logit."""
    return np.argmax(logits, axis=1).astype(np.int32)


def top2_margin(logits):
    """top-1 minus top-2 logit per image (float64)."""
    s = np.sort(logits.astype(np.float64), axis=1)
    return s[:, -1] - s[:, -2]


def eval_schemes(arch, bank, schemes, x, labels, chunk=256):
    """Per scheme: (accuracy, correct count, predictions, margins)."""
    accs, counts, preds, margins = [], [], [], []
    for scheme in schemes:
        lg = forward_scheme(arch, bank, scheme, x, chunk)
        p = predict(lg)
        c = int(np.sum(p == labels))
        accs.append(c / len(labels))
        counts.append(c)
        preds.append(p)
        margins.append(top2_margin(lg))
    return np.asarray(accs), np.asarray(counts, dtype=np.int64), np.stack(preds), np.stack(margins)


# ----------------------------------------------------------------------------
# Analytic global arithmetic intensity (Section 1 (i); Section 2.2 last paragraph)
# ----------------------------------------------------------------------------
def layer_shapes(arch):
    """Per layer: (K, Hin, Win, Hout, Wout) from the wiring."""
    shapes, hw = [], []
    for layer in arch["layers"]:
        if layer["input"] < 0:
            hi, wi = arch["in_h"], arch["in_w"]
        else:
            hi, wi = hw[layer["input"]]
        if layer["kind"] == "fc":
            shapes.append((layer["cin"], 1, 1, 1, 1))
            hw.append((1, 1))
            continue
        ho = out_hw(hi, layer["k"], layer["stride"], layer["pad"])
        wo = out_hw(wi, layer["k"], layer["stride"], layer["pad"])
        cin_g = 1 if layer["kind"] == "dw" else layer["cin"]
        shapes.append((cin_g * layer["k"] ** 2, hi, wi, ho, wo))
        hw.append((ho, wo))
    return shapes


def scheme_ai(arch, scheme, batch=1):
    """AI(q) = sum_l FLOPs_l / sum_l Bytes_l(q_l), in FLOP per byte.

    The paper says AI is computed "analytically from FLOPs and memory traffic" and gives
    no formula.  Reading: per weight layer (conv, depthwise, projection, classifier)
      FLOPs_l = 2 * cout * K * Ho * Wo * batch
      Bytes_l = cout * K * q_l / 8  +  4 * batch * (cin * Hi * Wi + cout * Ho * Wo)
    Biases, scales, batch-norm, activations, residual adds and pooling count for nothing.
    Returns (ai, flops, bytes) as Python floats.
    """
    flops = 0.0
    nbytes = 0.0
    for layer, (K, hi, wi, ho, wo), bits in zip(arch["layers"], layer_shapes(arch), scheme):
        if int(bits) not in ALLOWED_BITS:
            raise ValueError(f"unsupported bit-width {bits}")
        flops += 2.0 * layer["cout"] * K * ho * wo * batch
        nbytes += layer["cout"] * K * int(bits) / 8.0
        nbytes += 4.0 * batch * (layer["cin"] * hi * wi + layer["cout"] * ho * wo)
    return flops / nbytes, flops, nbytes


# ----------------------------------------------------------------------------
# AIQ objective and the two searches (Section 2.1, Section 2.2)
# ----------------------------------------------------------------------------
def aiq_loss(ai, acc, acc_fp, lam):
    """L(q; lambda) = -lambda * AI(q) + (1 - lambda) * AccLoss(q)   (Section 2.1).

    The paper does not state the units of AccLoss nor a normalisation of AI.  Reading:
    AccLoss(q) = 100 * (acc(q_FP) - acc(q)) in percentage points, AI in FLOP per byte,
    neither normalised.  Parity unpinned for this choice of units (nothing printed in the
    paper fixes it); the search logic around it is pinned by hand-worked tables.
    """
    return -lam * ai + (1.0 - lam) * 100.0 * (acc_fp - acc)


def greedy_search(n_layers, acc_fn, ai_fn, lam, options=(8, 4), layers=None):
    """Greedy search of Section 2.2.

    Start from the all-FP32 scheme.  At each iteration the candidate moves are "lower the
    bit-width of a still unquantized (32-bit) layer i to b", for every selectable layer i
    and every b in `options`; the move with the smallest Delta L = L(candidate) - L(current)
    is taken when that Delta L is negative.  As many iterations as there are selectable
    layers.  Ties go to the first candidate in (layer, option) order.  When no move improves
    the loss the scheme can no longer change and the remaining iterations are no-ops.
    acc_fn(schemes [S][L] uint8) -> accuracies [S]; ai_fn(scheme) -> AI.
    Returns (scheme, trace) with trace = list of (layer, bits, accepted, loss_after).
    """
    layers = list(range(n_layers)) if layers is None else list(layers)
    q = np.full(n_layers, 32, np.uint8)
    acc_fp = float(acc_fn(q[None, :])[0])
    cur = aiq_loss(ai_fn(q), acc_fp, acc_fp, lam)
    trace = []
    for _ in range(len(layers)):
        moves = [(i, b) for i in layers if q[i] == 32 for b in options if b < 32]
        if not moves:
            break
        cands = np.repeat(q[None, :], len(moves), axis=0)
        for r, (i, b) in enumerate(moves):
            cands[r, i] = b
        accs = acc_fn(cands)
        best, best_delta = -1, 0.0
        for r in range(len(moves)):
            delta = aiq_loss(ai_fn(cands[r]), float(accs[r]), acc_fp, lam) - cur
            if best < 0 or delta < best_delta:
                best, best_delta = r, delta
        i, b = moves[best]
        if best_delta < 0:
            q = cands[best].copy()
            cur = cur + best_delta
            trace.append((i, b, 1, cur))
        else:
            trace.append((i, b, 0, cur))
            break
    return q, trace


def coordinate_descent(n_layers, acc_fn, ai_fn, lam, options=(32, 8, 4), layers=None, max_passes=8):
    """Coordinate descent of Section 2.2.

    Start from the all-FP32 scheme.  Visit the selectable layers in order; for each, hold
    the others fixed and set q_i to the b in `options` with the smallest L (the current
    value stays on ties; among strictly better values the first in option order wins).
    Repeat passes until a pass changes nothing (or `max_passes`).
    Returns (scheme, trace) with trace = list of (layer, bits, changed, loss_after).
    """
    layers = list(range(n_layers)) if layers is None else list(layers)
    q = np.full(n_layers, 32, np.uint8)
    acc_fp = float(acc_fn(q[None, :])[0])
    cur = aiq_loss(ai_fn(q), acc_fp, acc_fp, lam)
    trace = []
    for _ in range(max_passes):
        changed_any = False
        for i in layers:
            alts = [b for b in options if b != q[i]]
            cands = np.repeat(q[None, :], len(alts), axis=0)
            for r, b in enumerate(alts):
                cands[r, i] = b
            accs = acc_fn(cands)
            best, best_loss = -1, cur
            for r in range(len(alts)):
                loss = aiq_loss(ai_fn(cands[r]), float(accs[r]), acc_fp, lam)
                if loss < best_loss:
                    best, best_loss = r, loss
            if best >= 0:
                q = cands[best].copy()
                cur = best_loss
                changed_any = True
                trace.append((i, int(q[i]), 1, cur))
            else:
                trace.append((i, int(q[i]), 0, cur))
        if not changed_any:
            break
    return q, trace


# ----------------------------------------------------------------------------
# Standalone quantized linear layer
# ----------------------------------------------------------------------------
def qlinear(values, scales, bias, bits, x):
    """y[m,n] = sum_k w_hat[n,k] * x[m,k] (+ bias_n), float64 accumulate, float32 result."""
    w_hat = dequantize_rows(values, scales, bits).astype(np.float64)
    y = np.matmul(x.astype(np.float64), w_hat.T)
    if bias is not None:
        y = y + bias.astype(np.float64)
    return y.astype(np.float32)

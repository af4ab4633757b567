"""ctypes binding of libaiq.so: argument marshalling only.

Every function here has the name of the C entry point it calls (see include/aiq.h) and
does nothing but convert arguments: torch tensors supply device pointers and the current
stream, NumPy arrays supply host pointers.  All arithmetic runs inside the CUDA library;
if the library is missing the import of this module fails.
"""
import ctypes as C
import os

import numpy as np

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libaiq.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED_BITS, ERR_SHAPE, ERR_WORKSPACE_TOO_SMALL = 1, 2, 3, 4
ERR_CUDA, ERR_NOT_SM100, ERR_NONFINITE, ERR_TIMEOUT = 5, 6, 7, 8

LAYER_KIND = {"conv": 0, "dw": 1, "fc": 2}
ACT = {"none": 0, "relu": 1, "relu6": 2}

EXPORTS = [
    "aiq_status_string", "aiq_last_error", "aiq_fold_bn", "aiq_packed_row_bytes",
    "aiq_quantize_layer", "aiq_qlinear", "aiq_qlinear_workspace_bytes", "aiq_model_bytes", "aiq_model_create",
    "aiq_model_destroy", "aiq_model_num_layers", "aiq_model_num_classes",
    "aiq_model_layer_folded", "aiq_model_layer_packed", "aiq_workspace_bytes", "aiq_forward",
    "aiq_eval_schemes", "aiq_set_eval_options", "aiq_set_fusion", "aiq_set_small_pass_images", "aiq_quantize_layer_per_tensor", "aiq_set_scale_granularity", "aiq_last_call_stats", "aiq_scheme_ai",
    "aiq_profile_start", "aiq_profile_stop", "aiq_forward_static",
    "aiq_set_compute_path", "aiq_model_status", "aiq_debug_expire_wait", "aiq_search_greedy", "aiq_search_coordinate_descent",
]

PATH_AUTO, PATH_FP32, PATH_TENSOR, PATH_TENSOR_TILES = 0, 1, 2, 3

STATIC_WORKSPACE_BYTES = 8 * 1024 * 1024

KERNEL_KINDS = ["fold", "quantize", "qlinear", "conv", "depthwise", "pool", "argmax", "conv_tc"]


class AiqError(RuntimeError):
    def __init__(self, status, detail):
        super().__init__(f"aiq status {status} ({status_string(status)}): {detail}")
        self.status = status


class LayerDesc(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "cin", "cout", "ksize", "stride", "pad", "act",
                                         "input", "residual", "has_bn")]


class ArchDesc(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("in_c", C.c_int32), ("in_h", C.c_int32),
                ("in_w", C.c_int32), ("layers", C.POINTER(LayerDesc))]


class KernelProfile(C.Structure):
    _fields_ = [("launches", C.c_int64), ("ms", C.c_double), ("flops", C.c_double),
                ("bytes", C.c_double)]


class SearchStep(C.Structure):
    _fields_ = [("layer", C.c_int32), ("bits", C.c_int32), ("accepted", C.c_int32), ("candidates", C.c_int32),
                ("loss", C.c_double), ("acc", C.c_double), ("ai", C.c_double)]


class LayerWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("W", "gamma", "beta", "mean", "var", "bias")]


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with "
                          "`python -m paper_2512_14090_b200.build` (there is no fallback path)")
    lib = C.CDLL(_LIB_PATH)
    vp, i32, f32, sz = C.c_void_p, C.c_int, C.c_float, C.c_size_t
    lib.aiq_status_string.restype = C.c_char_p
    lib.aiq_status_string.argtypes = [i32]
    lib.aiq_last_error.restype = C.c_char_p
    lib.aiq_last_error.argtypes = []
    lib.aiq_fold_bn.restype = i32
    lib.aiq_fold_bn.argtypes = [vp, vp, vp, vp, vp, i32, i32, f32, vp, vp, vp]
    lib.aiq_packed_row_bytes.restype = sz
    lib.aiq_packed_row_bytes.argtypes = [i32, i32]
    lib.aiq_quantize_layer.restype = i32
    lib.aiq_quantize_layer.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    lib.aiq_qlinear.restype = i32
    lib.aiq_qlinear.argtypes = [vp, vp, vp, i32, i32, i32, vp, i32, vp, vp, sz, vp]
    lib.aiq_qlinear_workspace_bytes.restype = sz
    lib.aiq_qlinear_workspace_bytes.argtypes = [i32, i32, i32, i32]
    lib.aiq_model_bytes.restype = sz
    lib.aiq_model_bytes.argtypes = [C.POINTER(ArchDesc)]
    lib.aiq_model_create.restype = i32
    lib.aiq_model_create.argtypes = [C.POINTER(ArchDesc), C.POINTER(LayerWeights), vp, sz, vp,
                                     C.POINTER(vp)]
    lib.aiq_model_destroy.restype = None
    lib.aiq_model_destroy.argtypes = [vp]
    lib.aiq_model_num_layers.restype = i32
    lib.aiq_model_num_layers.argtypes = [vp]
    lib.aiq_model_num_classes.restype = i32
    lib.aiq_model_num_classes.argtypes = [vp]
    lib.aiq_model_layer_folded.restype = i32
    lib.aiq_model_layer_folded.argtypes = [vp, i32, C.POINTER(vp), C.POINTER(vp), C.POINTER(i32),
                                           C.POINTER(i32)]
    lib.aiq_model_layer_packed.restype = i32
    lib.aiq_model_layer_packed.argtypes = [vp, i32, i32, C.POINTER(vp), C.POINTER(vp)]
    lib.aiq_workspace_bytes.restype = sz
    lib.aiq_workspace_bytes.argtypes = [vp, i32, i32]
    lib.aiq_forward.restype = i32
    lib.aiq_forward.argtypes = [vp, vp, vp, i32, vp, vp, sz, vp]
    lib.aiq_eval_schemes.restype = i32
    lib.aiq_eval_schemes.argtypes = [vp, vp, i32, vp, vp, i32, vp, vp, vp, vp, sz, vp]
    lib.aiq_set_eval_options.restype = None
    lib.aiq_set_eval_options.argtypes = [i32, i32]
    lib.aiq_quantize_layer_per_tensor.restype = i32
    lib.aiq_quantize_layer_per_tensor.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp]
    lib.aiq_set_scale_granularity.restype = None
    lib.aiq_set_scale_granularity.argtypes = [i32]
    lib.aiq_set_fusion.restype = None
    lib.aiq_set_fusion.argtypes = [i32, i32]
    lib.aiq_set_small_pass_images.restype = None
    lib.aiq_set_small_pass_images.argtypes = [i32]
    lib.aiq_last_call_stats.restype = None
    lib.aiq_last_call_stats.argtypes = [C.POINTER(C.c_int64)] * 3
    lib.aiq_search_greedy.restype = i32
    lib.aiq_search_greedy.argtypes = [vp, vp, i32, vp, i32, C.c_double, vp, vp, i32, vp,
                                      C.POINTER(SearchStep), i32, C.POINTER(C.c_int), vp, sz, vp]
    lib.aiq_search_coordinate_descent.restype = i32
    lib.aiq_search_coordinate_descent.argtypes = [vp, vp, i32, vp, i32, C.c_double, i32, vp, vp, i32, vp,
                                                  C.POINTER(SearchStep), i32, C.POINTER(C.c_int), vp, sz, vp]
    lib.aiq_scheme_ai.restype = i32
    lib.aiq_scheme_ai.argtypes = [vp, vp, i32, C.POINTER(C.c_double), C.POINTER(C.c_double),
                                  C.POINTER(C.c_double)]
    lib.aiq_forward_static.restype = i32
    lib.aiq_forward_static.argtypes = [vp, vp, vp, i32, vp, vp]
    lib.aiq_model_status.restype = i32
    lib.aiq_model_status.argtypes = [vp, vp]
    lib.aiq_debug_expire_wait.restype = i32
    lib.aiq_debug_expire_wait.argtypes = [vp, C.c_int64, vp]
    lib.aiq_set_compute_path.restype = None
    lib.aiq_set_compute_path.argtypes = [i32]
    lib.aiq_profile_start.restype = i32
    lib.aiq_profile_start.argtypes = []
    lib.aiq_profile_stop.restype = i32
    lib.aiq_profile_stop.argtypes = [C.POINTER(KernelProfile)]
    return lib


lib = _load()


def status_string(status):
    return lib.aiq_status_string(int(status)).decode()


def last_error():
    return lib.aiq_last_error().decode()


def _check(status):
    if status != OK:
        raise AiqError(status, last_error())


def _dev(t):
    """Device pointer of a contiguous CUDA tensor (None -> NULL)."""
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("expected a contiguous CUDA tensor")
    return C.c_void_p(t.data_ptr())


def _host(a):
    return C.c_void_p(a.ctypes.data) if a is not None else None


def _stream(stream=None):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return C.c_void_p(s.cuda_stream)


def arch_desc(arch):
    """(ArchDesc, keep-alive list) from an architecture dict (kind/cin/cout/k/...)."""
    layers = (LayerDesc * len(arch["layers"]))()
    for d, l in zip(layers, arch["layers"]):
        d.kind, d.cin, d.cout, d.ksize = LAYER_KIND[l["kind"]], l["cin"], l["cout"], l["k"]
        d.stride, d.pad, d.act = l["stride"], l["pad"], ACT[l["act"]]
        d.input, d.residual, d.has_bn = l["input"], l["residual"], int(bool(l["has_bn"]))
    desc = ArchDesc(len(arch["layers"]), arch["in_c"], arch["in_h"], arch["in_w"], layers)
    return desc, layers


# ------------------------------------------------------------------------- plain calls
def aiq_packed_row_bytes(K, bits):
    return int(lib.aiq_packed_row_bytes(int(K), int(bits)))


def aiq_fold_bn(W, gamma, beta, mean, var, Wf, bf, eps=1e-5, stream=None):
    N = W.shape[0]
    K = W.numel() // N
    _check(lib.aiq_fold_bn(_dev(W), _dev(gamma), _dev(beta), _dev(mean), _dev(var), N, K,
                           C.c_float(eps), _dev(Wf), _dev(bf), _stream(stream)))


def aiq_quantize_layer(W, bits, packed_out, scales_out, nonfinite_flag=None, stream=None):
    N, K = W.shape
    _check(lib.aiq_quantize_layer(_dev(W), N, K, int(bits), _dev(packed_out), _dev(scales_out),
                                  _dev(nonfinite_flag), _stream(stream)))


def aiq_qlinear_workspace_bytes(N, K, bits, M):
    return int(lib.aiq_qlinear_workspace_bytes(int(N), int(K), int(bits), int(M)))


def aiq_qlinear(packed, scales, bias, N, K, bits, x, y, workspace=None, stream=None):
    M = x.shape[0]
    _check(lib.aiq_qlinear(_dev(packed), _dev(scales), _dev(bias), int(N), int(K), int(bits),
                           _dev(x), int(M), _dev(y), _dev(workspace),
                           workspace.numel() if workspace is not None else 0, _stream(stream)))


def aiq_set_eval_options(chunk=0, share_prefix=True):
    lib.aiq_set_eval_options(int(chunk), int(bool(share_prefix)))


SCALE_PER_CHANNEL, SCALE_PER_TENSOR = 0, 1


def aiq_set_scale_granularity(granularity):
    lib.aiq_set_scale_granularity(int(granularity))


def aiq_quantize_layer_per_tensor(W, bits, packed_out, scales_out, scratch, nonfinite_flag=None, stream=None):
    N, K = W.shape
    _check(lib.aiq_quantize_layer_per_tensor(_dev(W), int(N), int(K), int(bits), _dev(packed_out), _dev(scales_out),
                                             _dev(nonfinite_flag), _dev(scratch), _stream(stream)))


def aiq_set_fusion(blocks=True, pool=True, inverted_residual="auto"):
    """inverted_residual: "auto" (fuse where measured faster), True (every eligible block), False."""
    ir = 4 if inverted_residual == "auto" else (2 if inverted_residual else 0)
    lib.aiq_set_fusion(int(bool(blocks)) | ir, int(bool(pool)))


def aiq_set_small_pass_images(image_schemes):
    lib.aiq_set_small_pass_images(int(image_schemes))


def aiq_set_compute_path(path):
    lib.aiq_set_compute_path(int(path))


def aiq_last_call_stats():
    a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
    lib.aiq_last_call_stats(C.byref(a), C.byref(b), C.byref(c))
    return dict(kernel_launches=a.value, layer_evals=b.value, layer_evals_unshared=c.value)


def aiq_profile_start():
    _check(lib.aiq_profile_start())


def aiq_profile_stop():
    """{kind: dict(launches, ms, flops, bytes)} for the launches since aiq_profile_start."""
    out = (KernelProfile * len(KERNEL_KINDS))()
    _check(lib.aiq_profile_stop(out))
    return {k: dict(launches=o.launches, ms=o.ms, flops=o.flops, bytes=o.bytes)
            for k, o in zip(KERNEL_KINDS, out)}


# ------------------------------------------------------------------------- model object
class Model:
    """Owns the device memory the C model lives in (a torch uint8 tensor) and the handle."""

    def __init__(self, arch, params, device="cuda:0", stream=None, mem=None):
        """Uploads `params` (host float32 arrays), folds and builds the weight bank.
        `mem`: an existing uint8 CUDA tensor to build into (reused across rebuilds)."""
        import torch
        self.arch = arch
        self.device = torch.device(device)
        desc, self._keep_layers = arch_desc(arch)
        self._desc = desc
        nbytes = int(lib.aiq_model_bytes(C.byref(desc)))
        if nbytes == 0:
            raise AiqError(ERR_INVALID_ARG, last_error())
        if mem is not None and mem.numel() >= nbytes:
            self.mem = mem
        else:
            self.mem = torch.empty(nbytes, dtype=torch.uint8, device=self.device)
        weights = (LayerWeights * len(params))()
        keep = []
        for w, p in zip(weights, params):
            for name in ("W", "gamma", "beta", "mean", "var", "bias"):
                if name in p and p[name] is not None:
                    a = np.ascontiguousarray(p[name], dtype=np.float32)
                    keep.append(a)
                    setattr(w, name, a.ctypes.data)
        handle = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(lib.aiq_model_create(C.byref(desc), weights, _dev(self.mem), self.mem.numel(),
                                        _stream(stream), C.byref(handle)))
        self.handle = handle
        self.n_layers = int(lib.aiq_model_num_layers(handle))
        self.n_classes = int(lib.aiq_model_num_classes(handle))
        self._ws = None

    def close(self):
        if getattr(self, "handle", None) and lib is not None:      # lib is None at interpreter exit
            lib.aiq_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        self.close()

    # views for inspection --------------------------------------------------------
    def layer_folded(self, layer):
        """(Wf [N][K], bias [N]) as torch views into the model memory."""
        wf, b, n, k = C.c_void_p(), C.c_void_p(), C.c_int(), C.c_int()
        _check(lib.aiq_model_layer_folded(self.handle, layer, C.byref(wf), C.byref(b), C.byref(n), C.byref(k)))
        return (self._view(wf.value, n.value * k.value * 4).view(dtype=_f32()).view(n.value, k.value),
                self._view(b.value, n.value * 4).view(dtype=_f32()))

    def layer_packed(self, layer, bits):
        wf, b, n, k = C.c_void_p(), C.c_void_p(), C.c_int(), C.c_int()
        _check(lib.aiq_model_layer_folded(self.handle, layer, C.byref(wf), C.byref(b), C.byref(n), C.byref(k)))
        p, s = C.c_void_p(), C.c_void_p()
        _check(lib.aiq_model_layer_packed(self.handle, layer, int(bits), C.byref(p), C.byref(s)))
        rb = aiq_packed_row_bytes(k.value, bits)
        return (self._view(p.value, n.value * rb).view(n.value, rb),
                self._view(s.value, n.value * 4).view(dtype=_f32()))

    def _view(self, ptr, nbytes):
        off = ptr - self.mem.data_ptr()
        assert 0 <= off and off + nbytes <= self.mem.numel()
        return self.mem[off:off + nbytes]

    # workspace -------------------------------------------------------------------
    def aiq_workspace_bytes(self, max_batch, max_schemes):
        return int(lib.aiq_workspace_bytes(self.handle, int(max_batch), int(max_schemes)))

    def workspace(self, max_batch, max_schemes):
        import torch
        need = self.aiq_workspace_bytes(max_batch, max_schemes)
        if self._ws is None or self._ws.numel() < need:
            self._ws = None
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    # the calls -------------------------------------------------------------------
    def aiq_forward(self, scheme_bits, x, logits=None, workspace=None, stream=None):
        import torch
        scheme = np.ascontiguousarray(scheme_bits, dtype=np.uint8)
        if scheme.shape != (self.n_layers,):
            raise ValueError("scheme length must equal the number of layers")
        B = x.shape[0]
        if logits is None:
            logits = torch.empty((B, self.n_classes), dtype=torch.float32, device=self.device)
        ws = workspace if workspace is not None else self.workspace(B, 1)
        _check(lib.aiq_forward(self.handle, _host(scheme), _dev(x), B, _dev(logits), _dev(ws),
                               ws.numel(), _stream(stream)))
        return logits

    def aiq_forward_static(self, scheme_bits, x, logits, stream=None):
        """aiq_forward on the library's built-in workspace.  `logits` must be provided by the
        caller ([batch][n_classes] float32 CUDA tensor): this call allocates nothing."""
        scheme = np.ascontiguousarray(scheme_bits, dtype=np.uint8)
        if scheme.shape != (self.n_layers,):
            raise ValueError("scheme length must equal the number of layers")
        _check(lib.aiq_forward_static(self.handle, _host(scheme), _dev(x), int(x.shape[0]),
                                      _dev(logits), _stream(stream)))
        return logits

    def aiq_eval_schemes(self, schemes, x, labels, preds=None, workspace=None, chunk=1024,
                         stream=None):
        schemes = np.ascontiguousarray(schemes, dtype=np.uint8)
        if schemes.ndim != 2 or schemes.shape[1] != self.n_layers:
            raise ValueError("schemes must be [S][L]")
        S, N = schemes.shape[0], x.shape[0]
        acc = np.zeros(S, dtype=np.float32)
        counts = np.zeros(S, dtype=np.int32)
        ws = workspace if workspace is not None else self.workspace(min(chunk, N), S)
        _check(lib.aiq_eval_schemes(self.handle, _host(schemes), S, _dev(x), _dev(labels), N,
                                    _host(acc), _host(counts), _dev(preds), _dev(ws), ws.numel(),
                                    _stream(stream)))
        return acc, counts

    def _search(self, which, x, labels, lam, options, layers, max_passes, workspace, chunk, stream):
        options = np.ascontiguousarray(options, dtype=np.uint8)
        n_sel = self.n_layers if layers is None else len(layers)
        lay = None if layers is None else np.ascontiguousarray(layers, dtype=np.int32)
        N = x.shape[0]
        ws = workspace if workspace is not None else self.workspace(min(chunk, N), max(1, n_sel * len(options)))
        scheme = np.zeros(self.n_layers, dtype=np.uint8)
        cap = 4 * (n_sel + 1) * max(1, max_passes)
        trace = (SearchStep * cap)()
        n_trace = C.c_int(0)
        if which == "greedy":
            _check(lib.aiq_search_greedy(self.handle, _host(lay), n_sel, _host(options), len(options), float(lam),
                                         _dev(x), _dev(labels), N, _host(scheme), trace, cap, C.byref(n_trace),
                                         _dev(ws), ws.numel(), _stream(stream)))
        else:
            _check(lib.aiq_search_coordinate_descent(self.handle, _host(lay), n_sel, _host(options), len(options),
                                                     float(lam), int(max_passes), _dev(x), _dev(labels), N,
                                                     _host(scheme), trace, cap, C.byref(n_trace), _dev(ws),
                                                     ws.numel(), _stream(stream)))
        steps = [dict(layer=t.layer, bits=t.bits, accepted=t.accepted, candidates=t.candidates, loss=t.loss,
                      acc=t.acc, ai=t.ai) for t in trace[:min(n_trace.value, cap)]]
        return scheme, steps

    def aiq_search_greedy(self, x, labels, lam, options=(8, 4), layers=None, workspace=None, chunk=1024,
                          stream=None):
        return self._search("greedy", x, labels, lam, options, layers, 1, workspace, chunk, stream)

    def aiq_search_coordinate_descent(self, x, labels, lam, options=(32, 8, 4), layers=None, max_passes=8,
                                      workspace=None, chunk=1024, stream=None):
        return self._search("cd", x, labels, lam, options, layers, max_passes, workspace, chunk, stream)

    def aiq_model_status(self, stream=None):
        _check(lib.aiq_model_status(self.handle, _stream(stream)))

    def aiq_debug_expire_wait(self, limit_cycles, stream=None):
        _check(lib.aiq_debug_expire_wait(self.handle, int(limit_cycles), _stream(stream)))

    def aiq_scheme_ai(self, scheme_bits, ai_batch=1):
        scheme = np.ascontiguousarray(scheme_bits, dtype=np.uint8)
        if scheme.shape != (self.n_layers,):
            raise ValueError("scheme length must equal the number of layers")
        ai, fl, by = C.c_double(), C.c_double(), C.c_double()
        _check(lib.aiq_scheme_ai(self.handle, _host(scheme), int(ai_batch), C.byref(ai), C.byref(fl),
                                 C.byref(by)))
        return ai.value, fl.value, by.value


def _f32():
    import torch
    return torch.float32

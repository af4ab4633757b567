#!/usr/bin/env python
"""Benchmark of the AIQ scheme-evaluation hot path on B200.

One step = one greedy search step on CIFAR ResNet-20: build the model's weight bank (fold
batch-norm, quantize + pack every layer at 4/8/16/32 bits), then score 21 candidate schemes
(each lowers one conv layer of an all-8-bit scheme to 4 bits) on a 10,000-image evaluation
set, and compute each candidate's analytic arithmetic intensity.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]

Prints one JSON line (rank 0).  `value` is scheme evaluations per second with the images
resident in device memory; `e2e` repeats the measurement with the images in pinned host
memory, copied to the device inside the timed region.  With N > 1 (torchrun) every rank
scores the same candidates on its own 10,000-image shard and the per-scheme counts are
summed over ranks (weak scaling).
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

N_IMAGES = 10000
SEED_MODEL, SEED_IMAGES = 1234, 5679
WORKLOAD = "resnet20_cifar_greedy_step: 21 schemes (all-8, one conv layer -> 4 bits) x 10000 images"
METRIC = "scheme evals/sec (ResNet-20, 10k imgs)"
UNIT = "scheme-evals/s"
# images per evaluator pass of the headline workload: two passes over the 10,000 images (a pass
# costs ~26 launches with their set-up; fewer, larger passes amortise it)
DEFAULT_CHUNK = 5008


def eval_workload(name):
    """The two scheme-sweep workloads: what is evaluated, on what, and how the oracle samples it."""
    from aiq_workloads import (resnet20, mobilenet_v2, one_layer_lowered_schemes, coordinate_step_schemes,
                               conv_layer_indices)
    if name == "resnet20_step":
        arch = resnet20()
        return dict(arch=arch, seed_model=SEED_MODEL, seed_images=SEED_IMAGES, n_images=N_IMAGES, image=(3, 32, 32),
                    schemes=one_layer_lowered_schemes(len(arch["layers"]), conv_layer_indices(arch)),
                    chunk=DEFAULT_CHUNK, workload=WORKLOAD, metric=METRIC, oracle_images=128, ref_images=16,
                    tc_kernel="conv_rs_kernel (tcgen05 bf16, fp32 accumulate, row-streaming)")
    if name == "mbv2_imagenet_cd_step":
        # one coordinate-descent sweep slice (Section 2.2): 52 candidates, each moving one conv layer of
        # an all-8 scheme to 32, 16 or 4 bits, on 2,048 ImageNet-shaped images
        arch = mobilenet_v2("imagenet")
        return dict(arch=arch, seed_model=4234, seed_images=4237, n_images=2048, image=(3, 224, 224),
                    schemes=coordinate_step_schemes(len(arch["layers"]), conv_layer_indices(arch)),
                    chunk=32, workload="mobilenet_v2_imagenet_coordinate_step: 52 schemes (all-8, one conv layer -> "
                                       "32 / 16 / 4 bits) x 2048 images of 3x224x224",
                    metric="scheme evals/sec (MobileNetV2-ImageNet, 2048 imgs)", oracle_images=2, ref_images=1,
                    tc_kernel="conv_pw_tc_kernel / conv_tc_kernel (tcgen05 bf16, fp32 accumulate)")
    raise ValueError(name)

# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel from one ncu
# capture, per image of the evaluator pass (traffic grows in proportion to the images of a launch;
# the capture runs a smaller pass than the benchmark).  None until captured / after the kernel changed.
NCU_TRAFFIC_BYTES_PER_LAUNCH_PER_IMAGE = 0.629e6
NCU_TRAFFIC_NOTE = ("dram__bytes_read.sum + dram__bytes_write.sum of the 15 row-streaming launches of one evaluator pass, "
                    "captured at 512 images per pass and scaled to this run's pass size by the images per launch")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=p["hbm_gbs"], bf16_tflops=p["bf16_tflops"],
                    bf16_tflops_sustained=p.get("bf16_tflops_sustained", p["bf16_tflops"]),
                    sm_max_mhz=p.get("sm_max_mhz", 1965.0), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                sm_max_mhz=1965.0, source="fallback")


class ClockSampler:
    """nvidia-smi sampling of SM clock and throttle reasons while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "100", "-i", str(self.gpu_index)], stdout=self.out, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1]))
                    mx.append(float(parts[2]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["no samples"])
        return dict(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons),
                    samples=len(sm))


def oracle_sample_rate(n_sample_images, schemes, arch, params, x, n_images=N_IMAGES):
    """Times the CPU oracle, as it stands, on `n_sample_images` images x all schemes and
    scales linearly to the `n_images`-image set.  Returns (scheme-evals/s, seconds, threads)."""
    from oracle import aiq_oracle as O
    threads = os.cpu_count() or 1
    try:
        from threadpoolctl import threadpool_info
        nt = [i.get("num_threads", 0) for i in threadpool_info() if i.get("user_api") == "blas"]
        if nt:
            threads = max(nt)
    except Exception:
        pass
    t0 = time.perf_counter()
    folded = O.fold_model(arch, params)
    bank = O.build_weight_bank(folded, bits_set=tuple(sorted({int(b) for b in np.unique(schemes)} | {8})))
    xs = x[:n_sample_images]
    labels = O.predict(O.forward_scheme(arch, bank, [8] * len(arch["layers"]), xs))
    O.eval_schemes(arch, bank, schemes, xs, labels)
    for s in schemes:
        O.scheme_ai(arch, s)
    dt = time.perf_counter() - t0
    evals_per_s = len(schemes) / (dt * (n_images / float(n_sample_images)))
    return evals_per_s, dt, threads


def run_reference(args, rank, world):
    """--impl reference: the CPU oracle on the host cores, rank 0 only."""
    if rank != 0:
        return
    from aiq_workloads import gen_model, gen_images
    wl = eval_workload(args.workload if args.workload == "mbv2_imagenet_cd_step" else "resnet20_step")
    arch, schemes, n_images = wl["arch"], wl["schemes"], wl["n_images"]
    params = gen_model(arch, wl["seed_model"])
    n_sample = wl["ref_images"]
    x = gen_images(n_sample, *wl["image"], wl["seed_images"])
    for _ in range(args.warmup):
        oracle_sample_rate(min(4, n_sample), schemes[:2], arch, params, x, n_images)
    secs, threads = 0.0, 1
    for _ in range(args.steps):
        _, dt, threads = oracle_sample_rate(n_sample, schemes, arch, params, x, n_images)
        secs += dt
    value = len(schemes) * args.steps / (secs * (n_images / float(n_sample)))
    sample = (f"each step: all {len(schemes)} schemes on the first {n_sample} of the {n_images} images (fold, bank, "
              f"labels, forward, count, AI), scaled linearly by {n_images}/{n_sample}")
    line = dict(impl="reference", metric=wl["metric"], value=value, unit=UNIT, n_gpus=args.gpus, steps=args.steps,
                warmup=args.warmup, ms_per_step=1000.0 * secs / args.steps * (n_images / float(n_sample)),
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=wl["workload"], note="CPU oracle (NumPy float64), extrapolated from a sample"),
                cpu_baseline=dict(value=value, unit=UNIT, cores=threads, kind="oracle", sample=sample),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line), flush=True)


def time_launches(torch, fn, n):
    """ms per launch of fn(i), i = 0..n-1, replayed from a CUDA graph so that host launch
    overhead (about 10 us per call through ctypes) does not mask microsecond kernels."""
    for i in range(min(n, 4)):
        fn(i)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(n):
            fn(i)
    graph.replay()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    graph.replay()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n          # ms per launch


L2_ROTATE = 300e6       # operands rotate over copies totalling more than twice the L2 capacity


def measure_qlinear(aiq, torch, peaks, dev, N, K, bits_list, M_list, reps=20):
    """Standalone quantized linear layer against the HBM roofline (weights rotate through HBM)."""
    from aiq_workloads import gen_linear_case
    wh, _ = gen_linear_case(N, K, 1, 3234)
    w = torch.from_numpy(wh).to(dev)
    out = []
    for bits in bits_list:
        rb = aiq.aiq_packed_row_bytes(K, bits)
        packed0 = torch.empty((N, rb), dtype=torch.uint8, device=dev)
        scales = torch.empty(N, dtype=torch.float32, device=dev)
        aiq.aiq_quantize_layer(w, bits, packed0, scales)
        copies = max(2, int(np.ceil(L2_ROTATE / (N * rb))))
        packs = [packed0] + [packed0.clone() for _ in range(copies - 1)]
        for M in M_list:
            x = torch.randn((M, K), device=dev)
            y = torch.empty((M, N), device=dev)
            nbytes = N * rb + 4 * N + 4 * M * (K + N)
            flops = 2.0 * M * N * K
            n = reps * copies if M <= 16 else max(copies, 8)
            wsb = aiq.aiq_qlinear_workspace_bytes(N, K, bits, M)
            wsp = torch.empty(wsb, dtype=torch.uint8, device=dev) if wsb else None
            ms = time_launches(torch, lambda i: aiq.aiq_qlinear(packs[i % copies], scales, None, N, K, bits, x, y,
                                                                workspace=wsp), n)
            gbs = nbytes / (ms * 1e-3) / 1e9
            out.append(dict(workload="qlinear", N=N, K=K, bits=bits, M=M, us=ms * 1e3,
                            algorithmic_bytes=nbytes, GBps=gbs, frac_of_measured_hbm=gbs / peaks["hbm_gbs"],
                            frac_of_8TBps=gbs / 8000.0, TFLOPs=flops / (ms * 1e-3) / 1e12,
                            l2="weights rotate over %d copies" % copies))
    return out


def measure_quantize(aiq, torch, peaks, dev, N, K, bits_list, reps=20):
    """Quantize + pack kernel against the HBM roofline (the input rotates through HBM)."""
    w = torch.randn((N, K), device=dev) * 0.02
    copies = max(2, int(np.ceil(L2_ROTATE / (N * K * 4))))
    ws = [w] + [w.clone() for _ in range(copies - 1)]
    out = []
    for bits in bits_list:
        rb = aiq.aiq_packed_row_bytes(K, bits)
        packed = torch.empty((N, rb), dtype=torch.uint8, device=dev)
        scales = torch.empty(N, dtype=torch.float32, device=dev)
        nbytes = N * K * 4 + N * rb + N * 4
        ms = time_launches(torch, lambda i: aiq.aiq_quantize_layer(ws[i % copies], bits, packed, scales), reps * copies)
        gbs = nbytes / (ms * 1e-3) / 1e9
        out.append(dict(workload="quantize", N=N, K=K, bits=bits, us=ms * 1e3, algorithmic_bytes=nbytes,
                        GBps=gbs, frac_of_measured_hbm=gbs / peaks["hbm_gbs"], frac_of_8TBps=gbs / 8000.0,
                        l2="input rotates over %d copies" % copies))
    return out


def measure_mobilenet_layers(aiq, torch, peaks, dev, batch=256):
    """Depthwise and pointwise layers of MobileNetV2-CIFAR at `batch` (10 conv layers at 4 bits, the
    rest at 8): summed kernel time per kind from the library's per-launch events, against the
    algorithmic activation + weight bytes of those launches."""
    from aiq_workloads import mobilenet_v2, gen_model, mixed_int4_int8_scheme, conv_layer_indices
    arch = mobilenet_v2("cifar")
    model = aiq.Model(arch, gen_model(arch, 2234), device=dev)
    scheme = mixed_int4_int8_scheme(len(arch["layers"]), conv_layer_indices(arch), 10, 43)
    xb = torch.randn((batch, 3, 32, 32), device=dev)
    logits = torch.empty((batch, model.n_classes), device=dev)
    wsb = torch.empty(model.aiq_workspace_bytes(batch, 1), dtype=torch.uint8, device=dev)
    for _ in range(3):
        model.aiq_forward(scheme, xb, logits=logits, workspace=wsb)
    torch.cuda.synchronize()
    agg = {}
    reps = 5
    for _ in range(reps):
        aiq.aiq_profile_start()
        model.aiq_forward(scheme, xb, logits=logits, workspace=wsb)
        for k, v in aiq.aiq_profile_stop().items():
            a = agg.setdefault(k, dict(launches=0, ms=0.0, bytes=0.0, flops=0.0))
            for f in a:
                a[f] += v[f]
    model.close()
    out = []
    for kind, label in (("depthwise", "depthwise 3x3 layers (17)"), ("conv_tc", "pointwise 1x1 layers on tcgen05 (34)")):
        a = agg.get(kind)
        if not a or not a["launches"]:
            continue
        gbs = a["bytes"] / (a["ms"] * 1e-3) / 1e9
        out.append(dict(workload="mobilenet_v2_cifar_b%d" % batch, kernels=label, launches_per_forward=a["launches"] // reps,
                        us=a["ms"] * 1e3 / reps, algorithmic_bytes=a["bytes"] / reps, GBps=gbs,
                        frac_of_measured_hbm=gbs / peaks["hbm_gbs"], TFLOPs=a["flops"] / (a["ms"] * 1e-3) / 1e12))
    return out


def standalone_kernel_lines(aiq, torch, peaks, dev):
    """The `kernels` key of the headline line: the memory-bound kernels outside the headline step."""
    lines = measure_qlinear(aiq, torch, peaks, dev, 8192, 8192, (4, 8), (1, 4, 16, 256), reps=10)
    lines += measure_quantize(aiq, torch, peaks, dev, 8192, 8192, (4, 8, 16, 32), reps=5)
    lines += measure_mobilenet_layers(aiq, torch, peaks, dev)
    for ln in lines:
        for k, v in list(ln.items()):
            if isinstance(v, float):
                ln[k] = float("%.5g" % v)
    return lines


def run_kernel_sweep(args):
    """Standalone memory-bound kernels against the HBM roofline: the quantized linear layer
    (W [N][K] at 4/8/16/32 bits, M in {1,4,16,256}) and the quantize+pack kernel.  Operands
    rotate over enough distinct copies to exceed twice the L2 capacity, so every launch
    reads its weights from HBM.  One JSON line per case."""
    import torch
    from paper_2512_14090_b200 import build
    build.build()
    from paper_2512_14090_b200 import binding as aiq
    if args.fuse_inverted_residual or args.no_fuse_inverted_residual:
        aiq.aiq_set_fusion(True, True, inverted_residual=bool(args.fuse_inverted_residual))
    aiq.aiq_set_compute_path({"auto": aiq.PATH_AUTO, "tiles": aiq.PATH_TENSOR_TILES, "fp32": aiq.PATH_FP32}[args.path])
    from aiq_workloads import gen_linear_case
    peaks = measured_peaks()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    shapes = [(4096, 4096), (8192, 8192), (1280, 320)]
    if args.workload == "sensitivity":
        # the paper's single-layer study (Section 3, experiment 1; the 8b / 4b columns of Table 1):
        # every layer alone at 8 and at 4 bits, all others FP32, agreement with the FP32 model and AI
        from aiq_workloads import resnet20, gen_model, gen_images, one_layer_lowered_schemes
        arch = resnet20()
        model = aiq.Model(arch, gen_model(arch, SEED_MODEL), device=dev)
        L = model.n_layers
        x = torch.from_numpy(gen_images(N_IMAGES, 3, 32, 32, SEED_IMAGES)).to(dev)
        schemes = np.concatenate([np.full((1, L), 32, np.uint8),
                                  one_layer_lowered_schemes(L, list(range(L)), base=32, low=8),
                                  one_layer_lowered_schemes(L, list(range(L)), base=32, low=4)])
        ws = torch.empty(model.aiq_workspace_bytes(1024, len(schemes)), dtype=torch.uint8, device=dev)
        preds = torch.empty((len(schemes), N_IMAGES), dtype=torch.int32, device=dev)
        zeros = torch.zeros(N_IMAGES, dtype=torch.int32, device=dev)
        model.aiq_eval_schemes(schemes[:1], x, zeros, preds=preds[:1], workspace=ws)
        labels = preds[0].contiguous()
        model.aiq_eval_schemes(schemes, x, labels, workspace=ws)          # warm-up
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        acc, _ = model.aiq_eval_schemes(schemes, x, labels, workspace=ws)
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        ai = [model.aiq_scheme_ai(sc)[0] for sc in schemes]
        rows = [dict(layer=arch["layers"][i]["name"], acc_8b=float(acc[1 + i]), acc_4b=float(acc[1 + L + i]),
                     ai_8b=ai[1 + i], ai_4b=ai[1 + L + i]) for i in range(L)]
        print(json.dumps(dict(workload="sensitivity", model="resnet20", images=N_IMAGES, schemes=len(schemes),
                              seconds=dt, scheme_evals_per_s=len(schemes) / dt, ai_fp32=ai[0], layers=rows)), flush=True)
        model.close()
        return
    if args.workload == "search":
        # the two searches of Section 2.2 on ResNet-20 over the 10,000-image set (lambda = 0.9,
        # the paper's value): wall time of the whole search, every candidate scored by the evaluator
        from aiq_workloads import resnet20, gen_model, gen_images
        arch = resnet20()
        model = aiq.Model(arch, gen_model(arch, SEED_MODEL), device=dev)
        L = model.n_layers
        x = torch.from_numpy(gen_images(N_IMAGES, 3, 32, 32, SEED_IMAGES)).to(dev)
        ws = torch.empty(model.aiq_workspace_bytes(1024, 3 * L), dtype=torch.uint8, device=dev)
        preds = torch.empty((1, N_IMAGES), dtype=torch.int32, device=dev)
        model.aiq_eval_schemes(np.full((1, L), 32, np.uint8), x, torch.zeros(N_IMAGES, dtype=torch.int32, device=dev),
                               preds=preds, workspace=ws)
        labels = preds[0].contiguous()
        for name, fn in (("greedy", lambda: model.aiq_search_greedy(x, labels, 0.9, options=(8, 4), workspace=ws)),
                         ("coordinate_descent", lambda: model.aiq_search_coordinate_descent(
                             x, labels, 0.9, options=(32, 8, 4), max_passes=8, workspace=ws))):
            fn()                                                     # warm-up
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            scheme, steps = fn()
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            evals = 1 + sum(st["candidates"] for st in steps)
            print(json.dumps(dict(workload="search", algorithm=name, seconds=dt, scheme_evals=evals,
                                  scheme_evals_per_s=evals / dt, iterations=len(steps), images=N_IMAGES,
                                  final_scheme=[int(b) for b in scheme], final_ai=model.aiq_scheme_ai(scheme)[0],
                                  final_acc=steps[-1]["acc"] if steps else None, lam=0.9)), flush=True)
        model.close()
        return
    if args.workload == "forward":
        # one scheme, one batch, through aiq_forward (host plan + launches included): images/s
        from aiq_workloads import (resnet20, mobilenet_v2, gen_model, gen_images, gen_random_scheme,
                                   mixed_int4_int8_scheme, conv_layer_indices)
        cases = [("resnet20 (config 0)", resnet20(), 1234, [64], lambda a: gen_random_scheme(len(a["layers"]), 42)),
                 ("mobilenet_v2_cifar (config 2)", mobilenet_v2("cifar"), 2234, [1, 256],
                  lambda a: mixed_int4_int8_scheme(len(a["layers"]), conv_layer_indices(a), 10, 43)),
                 ("mobilenet_v2_imagenet (config 4)", mobilenet_v2("imagenet"), 4234, [1, 32, 256],
                  lambda a: np.full(len(a["layers"]), 8, np.uint8))]
        for name, arch, seed, batches, mk in cases:
            model = aiq.Model(arch, gen_model(arch, seed), device=dev)
            scheme = mk(arch)
            for B in batches:
                xb = torch.randn((B, arch["in_c"], arch["in_h"], arch["in_w"]), device=dev)
                logits = torch.empty((B, model.n_classes), device=dev)
                wsb = torch.empty(model.aiq_workspace_bytes(B, 1), dtype=torch.uint8, device=dev)
                for _ in range(3):
                    model.aiq_forward(scheme, xb, logits=logits, workspace=wsb)
                torch.cuda.synchronize()
                n = 20 if B <= 32 else 5
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(n):
                    model.aiq_forward(scheme, xb, logits=logits, workspace=wsb)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / n
                aiq.aiq_profile_start()
                model.aiq_forward(scheme, xb, logits=logits, workspace=wsb)
                kinds = {k: round(v["ms"], 4) for k, v in aiq.aiq_profile_stop().items() if v["launches"]}
                print(json.dumps(dict(workload="forward", model=name, batch=B, ms=ms, images_per_s=B / (ms * 1e-3),
                                      launches=aiq.aiq_last_call_stats()["kernel_launches"], kernel_ms=kinds)), flush=True)
            model.close()
        return
    if args.workload == "quantize":
        for (N, K) in shapes[:2]:
            for ln in measure_quantize(aiq, torch, peaks, dev, N, K, (4, 8, 16, 32)):
                print(json.dumps(ln), flush=True)
        return
    for (N, K) in shapes:
        for ln in measure_qlinear(aiq, torch, peaks, dev, N, K, (4, 8, 16, 32), (1, 4, 16, 256)):
            print(json.dumps(ln), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--chunk", type=int, default=0, help="images per evaluator pass (0 = library default)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernels", action="store_true", help="skip the standalone-kernel measurements of the headline line")
    ap.add_argument("--workload", default="resnet20_step", choices=["resnet20_step", "mbv2_imagenet_cd_step", "qlinear", "quantize", "forward", "search", "sensitivity"],
                    help="resnet20_step: the headline line (default).  mbv2_imagenet_cd_step: the coordinate-descent "
                         "sweep slice on ImageNet-shaped MobileNetV2 (52 candidates x 2,048 images), same line format.  "
                         "qlinear / quantize: per-case lines for the "
                         "standalone memory-bound kernels; forward: one scheme, one batch; search: the two searches "
                         "of Section 2.2 on ResNet-20; sensitivity: every layer alone at 8 / 4 bits from an FP32 "
                         "base (all 1 GPU)")
    ap.add_argument("--path", default="auto", choices=["auto", "tiles", "fp32"],
                    help="compute path of models created by the kernel workloads: auto (row-streaming tensor-core "
                         "kernels where the network allows), tiles (pixel-tile tensor-core kernels), fp32")
    ap.add_argument("--fuse-inverted-residual", action="store_true",
                    help="run every eligible inverted-residual block of MobileNetV2 as one kernel (aiq_set_fusion bit 1; "
                         "the default fuses a block only where that was measured faster)")
    ap.add_argument("--no-fuse-inverted-residual", action="store_true", help="never fuse inverted-residual blocks")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.workload not in ("resnet20_step", "mbv2_imagenet_cd_step"):
        if rank == 0:
            run_kernel_sweep(args)
        return
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist
    from paper_2512_14090_b200 import build
    build.build()
    from paper_2512_14090_b200 import binding as aiq          # fails loudly without libaiq.so
    if args.fuse_inverted_residual or args.no_fuse_inverted_residual:
        aiq.aiq_set_fusion(True, True, inverted_residual=bool(args.fuse_inverted_residual))
    from paper_2512_14090_b200.sharding import reduce_counts
    from aiq_workloads import gen_model, gen_images

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    wl = eval_workload(args.workload)
    arch, schemes, N_IMG = wl["arch"], wl["schemes"], wl["n_images"]
    params = gen_model(arch, wl["seed_model"])
    L = len(arch["layers"])
    S = len(schemes)
    x_host = torch.from_numpy(gen_images(N_IMG, *wl["image"], wl["seed_images"] + rank)).pin_memory()
    x_dev = x_host.to(dev)
    model = aiq.Model(arch, params, device=dev)
    chunk = args.chunk if args.chunk > 0 else wl["chunk"]
    aiq.aiq_set_eval_options(chunk, True)
    ws = torch.empty(model.aiq_workspace_bytes(chunk, S), dtype=torch.uint8, device=dev)

    # labels = arg-max of the FP32 model (the all-32 scheme), computed once by the library
    preds32 = torch.empty((1, N_IMG), dtype=torch.int32, device=dev)
    model.aiq_eval_schemes(np.full((1, L), 32, np.uint8), x_dev, torch.zeros(N_IMG, dtype=torch.int32, device=dev),
                           preds=preds32, workspace=ws)
    labels_dev = preds32[0].contiguous()
    labels_host = labels_dev.cpu().pin_memory()
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=dev)   # > L2 (126 MB)
    mem = model.mem
    launches = [0]
    bank_launches = sum(1 for l in arch["layers"] if l["has_bn"]) + L   # per layer: fold, one quantizer launch for the four widths
    result = {}

    def step(x, labels):
        m = aiq.Model(arch, params, device=dev, mem=mem)                 # fold + quantize bank
        acc, counts = m.aiq_eval_schemes(schemes, x, labels, workspace=ws)
        launches[0] += aiq.aiq_last_call_stats()["kernel_launches"] + bank_launches
        ai = [m.aiq_scheme_ai(s)[0] for s in schemes]
        if world > 1:
            counts, total, acc = reduce_counts(counts, N_IMG, device=dev)
        result.update(acc=np.asarray(acc, dtype=np.float64), ai=ai)
        m.close()

    def step_e2e():
        xd = x_dev_e2e.copy_(x_host, non_blocking=True)
        ld = labels_dev_e2e.copy_(labels_host, non_blocking=True)
        step(xd, ld)

    def timed(fn, n):
        total_ms = 0.0
        for _ in range(n):
            flush.zero_()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            total_ms += e0.elapsed_time(e1)
        return total_ms

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(ms):
        if world > 1:
            t = torch.tensor([ms], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            return float(t.item())
        return ms

    # ---- device-resident measurement ----------------------------------------------------
    for _ in range(args.warmup):
        step(x_dev, labels_dev)
    launches[0] = 0
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    aiq.aiq_profile_start()
    total_ms = timed(lambda: step(x_dev, labels_dev), args.steps)
    prof = aiq.aiq_profile_stop()
    barrier()
    clocks = sampler.stop()
    total_ms = max_over_ranks(total_ms)
    gpu_launches = launches[0]
    ms_per_step = total_ms / args.steps
    value = world * S * args.steps / (total_ms / 1000.0)

    # ---- end to end: images and labels start in pinned host memory ----------------------
    x_dev_e2e = torch.empty_like(x_dev)
    labels_dev_e2e = torch.empty_like(labels_dev)
    for _ in range(2):
        step_e2e()
    barrier()
    e2e_ms = max_over_ranks(timed(step_e2e, args.steps))
    barrier()
    weight_bytes = sum(int(np.asarray(v).nbytes) for p in params for v in p.values())
    h2d = x_host.numel() * 4 + labels_host.numel() * 4 + weight_bytes + S * L
    d2h = S * 4 + 4
    e2e_value = world * S * args.steps / (e2e_ms / 1000.0)

    # ---- roofline of the dominant kernel -------------------------------------------------
    peaks = measured_peaks()
    top = max(prof, key=lambda k: prof[k]["ms"])
    p = prof[top]
    avg_ms = p["ms"] / max(p["launches"], 1)
    sm_mhz = clocks.get("sm_mhz") or peaks["sm_max_mhz"]
    if top == "conv_tc":
        # tcgen05 implicit GEMM on activations stored as bfloat16 pairs.  Two rooflines apply:
        # the tensor pipe (algorithmic FLOPs = 2 per multiply-add of the convolution; the hi/lo
        # split doubles the MMA work, which is not counted) and HBM (algorithmic bytes = the input
        # and output tensors of every job plus the weights; at the default chunk a layer's tensors
        # of all candidate versions are far larger than L2, so they stream from and to DRAM).
        # The bound reported is the one with the larger fraction, i.e. the one that binds.
        t_s = p["ms"] / 1000.0
        tensor_achieved = p["flops"] / t_s / 1e12
        tensor_frac = tensor_achieved / peaks["bf16_tflops_sustained"]
        hbm_achieved = p["bytes"] / t_s / 1e9
        hbm_frac = hbm_achieved / peaks["hbm_gbs"]
        traffic = None
        if args.workload == "resnet20_step" and NCU_TRAFFIC_BYTES_PER_LAUNCH_PER_IMAGE is not None:
            traffic = NCU_TRAFFIC_BYTES_PER_LAUNCH_PER_IMAGE * min(chunk, N_IMG)
        common = dict(traffic=traffic, traffic_note=NCU_TRAFFIC_NOTE if traffic is not None else None,
                      kernel=wl["tc_kernel"],
                      launches=p["launches"], avg_launch_ms=avg_ms,
                      algorithmic_flops_per_launch=p["flops"] / max(p["launches"], 1),
                      algorithmic_bytes_per_launch=p["bytes"] / max(p["launches"], 1),
                      tensor_tflops=tensor_achieved, tensor_frac_of_sustained_bf16=tensor_frac,
                      hbm_gbs=hbm_achieved, hbm_frac_of_measured_copy=hbm_frac)
        if hbm_frac >= tensor_frac:
            roofline = dict(bound="hbm", achieved=hbm_achieved, peak=peaks["hbm_gbs"], unit="GB/s", frac=hbm_frac,
                            peak_source=f"HBM copy bandwidth, {peaks['source']}", **common)
        else:
            roofline = dict(bound="tensor", achieved=tensor_achieved, peak=peaks["bf16_tflops_sustained"],
                            unit="TFLOP/s", frac=tensor_frac,
                            peak_source=f"dense bf16 GEMM, sustained, {peaks['source']}", **common)
    elif top == "conv":
        # float32 multiply-add path: 148 SMs x 128 lanes x 2 FLOP per clock
        peak = 148 * 128 * 2 * sm_mhz * 1e6 / 1e12
        achieved = p["flops"] / (p["ms"] / 1000.0) / 1e12
        roofline = dict(bound="alu", achieved=achieved, peak=peak, unit="TFLOP/s", frac=achieved / peak,
                        traffic=None, kernel="conv_igemm_kernel (float32 FMA)",
                        peak_source=f"148 SMs x 128 FP32 lanes x 2 x {sm_mhz:.0f} MHz (median SM clock sampled during the run)",
                        launches=p["launches"], avg_launch_ms=avg_ms,
                        algorithmic_flops_per_launch=p["flops"] / max(p["launches"], 1),
                        algorithmic_bytes_per_launch=p["bytes"] / max(p["launches"], 1))
    else:
        achieved = p["bytes"] / (p["ms"] / 1000.0) / 1e9
        roofline = dict(bound="hbm", achieved=achieved, peak=peaks["hbm_gbs"], unit="GB/s",
                        frac=achieved / peaks["hbm_gbs"], traffic=None,
                        kernel=top, peak_source=f"HBM copy bandwidth, {peaks['source']}",
                        launches=p["launches"], avg_launch_ms=avg_ms,
                        algorithmic_bytes_per_launch=p["bytes"] / max(p["launches"], 1))
    all_ms = max(sum(q["ms"] for q in prof.values()), 1e-9)
    kernel_share = {k: round(v["ms"] / all_ms, 4) for k, v in prof.items() if v["launches"]}

    # ---- CPU oracle beside it (rank 0, N = 1 only) ----------------------------------------
    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_sample = wl["oracle_images"]
        v, dt, threads = oracle_sample_rate(n_sample, schemes, arch, params, x_host[:n_sample].numpy(), N_IMG)
        cpu_baseline = dict(value=v, unit=UNIT, cores=threads, kind="oracle", seconds=dt,
                            sample=f"all {S} schemes on the first {n_sample} of the {N_IMG} images (fold, bank, "
                                   f"labels, forward, count, AI), scaled linearly by {N_IMG}/{n_sample}")

    # ---- the memory-bound kernels outside the headline step (rank 0, N = 1 only) ------------
    kernels = None
    if rank == 0 and world == 1 and not args.no_kernels and args.workload == "resnet20_step":
        model.close()
        del ws, x_dev_e2e
        torch.cuda.empty_cache()
        kernels = standalone_kernel_lines(aiq, torch, peaks, dev)

    if rank == 0:
        line = dict(metric=wl["metric"], value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=args.warmup,
                    ms_per_step=ms_per_step, higher_is_better=True, scaling="weak", vs_baseline=None,
                    dtype="bf16", data="synthetic",
                    config=dict(workload=wl["workload"], images_per_rank=N_IMG, schemes=S, layers=L,
                                arithmetic="dense conv layers: bf16 tensor-core products of weight codes (or of two "
                                           "bfloat16 pieces of a 16-/32-bit weight) with activations held as hi + lo "
                                           "bfloat16 pairs, float32 accumulation; stem, depthwise, pooling and "
                                           "classifier in float32",
                                chunk=chunk, l2="flushed between timed steps (256 MiB write)",
                                step="fold + quantize bank (4/8/16/32 bits) + eval 21 schemes + AI",
                                labels="arg-max of the all-32-bit scheme, computed by the library",
                                prefix_sharing=True),
                    e2e=dict(value=e2e_value, unit=UNIT, h2d_bytes_per_step=h2d, d2h_bytes_per_step=d2h,
                             ms_per_step=e2e_ms / args.steps),
                    gpu_launches=gpu_launches, clocks=clocks, roofline=roofline, cpu_baseline=cpu_baseline,
                    kernel_time_share=kernel_share, kernels=kernels,
                    images_per_s=world * S * N_IMG * args.steps / (total_ms / 1000.0),
                    acc_min=float(result["acc"].min()), acc_max=float(result["acc"].max()),
                    ai_min=float(min(result["ai"])), ai_max=float(max(result["ai"])))
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

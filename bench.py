"""Benchmark of the VGG19 pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One "step" is one forward pass of the whole network on a batch of 100
224x224x3 bf16 images (the paper's headline shape, figure "Timings for the
VGG19 forward pass", N=100).  Rank 0 prints ONE JSON line: images/s with the
inputs resident in HBM (`value`), the same through the host-buffer entry point
with copies inside the timed region (`e2e`), the forward+backward throughput
(`fwd_bwd`) and that of a whole training step with the SGD update
(`train_step`), the roofline of the dominant kernel (the tensor-core
implicit-GEMM convolution on CTA pairs, timed per layer with CUDA events), the
achieved bandwidth of the largest memory-bound kernel (`hbm_bound`), and the
fp64 CPU checker timed on a bounded sample (`cpu_baseline`).

With N > 1 every rank runs the same batch-100 pass on its own GPU: the path
shards over the batch with no collective in the forward pass, so the aggregate
is N * 100 images per step over the slowest rank's time; the training step adds
its one exchange, an all-reduce of the gradients.  Under torchrun the ranks are
the launcher's; a plain `python bench.py --gpus N` (no WORLD_SIZE in the
environment) starts N ranks itself through torch.distributed.run.
`--backend gloo --dry` runs only the multi-rank plumbing (rendezvous, barrier,
max over ranks, gradient averaging, aggregation) on CPU ranks, for tests.

--impl reference times the CPU checker itself (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "VGG19 fwd images/s @batch 100, 224x224 bf16"
WORKLOAD = "configs[3]: full VGG19 forward, 224x224x3, batch 100, bf16 storage, fp32 accumulate"
H = W = 224
BATCH = 100
# Idle time after each kernel of the per-kernel timings: seven launches of one kernel are a millisecond or two of
# full load; without a pause the whole table runs as one stretch of tens of milliseconds and, on some boxes, at the
# power cap's clock, while the peaks it is compared with are burst figures taken on an idle GPU.
KERNEL_GAP_S = 0.05
CONV = [(224, 3, 64), (224, 64, 64), (112, 64, 128), (112, 128, 128), (56, 128, 256), (56, 256, 256),
        (56, 256, 256), (56, 256, 256), (28, 256, 512), (28, 512, 512), (28, 512, 512), (28, 512, 512),
        (14, 512, 512), (14, 512, 512), (14, 512, 512), (14, 512, 512)]
TRAIN_LR = 1e-6
FWD_FLOP_PER_IMAGE = sum(2 * s * s * co * 9 * ci for s, ci, co in CONV) + 2 * (25088 * 4096 + 4096 * 4096 + 4096 * 1000)


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples taken while the timed region runs."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self, t_begin=None, t_end=None, extra_window=None, kernel_window=None):
        """Summary of the samples taken between the two wall-clock times (all samples if none fall inside);
        with extra_window=(t0, t1) also {"extra": summary of the samples inside that second window}."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        import datetime
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                rows.append((ts, float(parts[1]), float(parts[2]),
                             [n for n, v in zip(names, parts[5:9]) if v.lower().startswith("active")]))
            except ValueError:
                continue
        self.file.close()
        os.unlink(self.file.name)
        def summary(t0, t1, label):
            inside = [r for r in rows if t0 is not None and t0 <= r[0] <= t1]
            use = inside if inside else rows
            reasons = sorted({n for r in use for n in r[3]})
            return {"sm_mhz": statistics.median(r[1] for r in use) if use else None,
                    "sm_max_mhz": max(r[2] for r in use) if use else None,
                    "samples": len(use), "window": label if inside else "whole run", "reasons": reasons}
        out = summary(t_begin, t_end, "timed region")
        if extra_window:
            out["extra"] = summary(extra_window[0], extra_window[1], "sustained region")
        if kernel_window:
            out["kernels"] = summary(kernel_window[0], kernel_window[1], "per-kernel timings")
        return out


TRAFFIC_PROFILE = os.path.join("profiles", "conv3x3_pair_tc_kernel_256_layer6_b48_full.txt")
TRAFFIC_SOURCES = ("tc_conv_pair.cu", "tc_common.cuh")


def kernel_source_digest():
    """sha256 over the source files of the dominant kernel: the ncu summary records the digest it was
    captured with, so that counters of an older kernel are not passed off as the current one's."""
    import hashlib
    h = hashlib.sha256()
    for name in TRAFFIC_SOURCES:
        with open(os.path.join(ROOT, "paper_1810_09868_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def dominant_kernel_traffic():
    """(bytes per batch-100 launch or None, note): dram__bytes_read.sum + dram__bytes_write.sum of the
    dominant kernel, read from its ncu summary under profiles/ (a layer-6 launch captured at the batch the
    file states) and scaled by the pixel count; None when the summary is missing, unreadable, or was
    captured with other kernel sources than the ones now in the tree."""
    import re
    path = os.path.join(ROOT, TRAFFIC_PROFILE)
    try:
        text = open(path).read()
    except OSError:
        return None, f"{TRAFFIC_PROFILE} missing"
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    total = 0.0
    for key in ("dram__bytes_read.sum", "dram__bytes_write.sum"):
        m = re.search(r"^" + re.escape(key) + r"\s+([0-9.]+)\s+(\w+)", text, re.M)
        if not m or m.group(2) not in unit:
            return None, f"{key} not found in {TRAFFIC_PROFILE}"
        total += float(m.group(1)) * unit[m.group(2)]
    b = re.search(r"^capture batch:\s*(\d+)", text, re.M)
    d = re.search(r"^kernel source digest:\s*(\w+)", text, re.M)
    if not b or not d:
        return None, f"{TRAFFIC_PROFILE} states no capture batch / source digest"
    if d.group(1) != kernel_source_digest():
        return None, "the kernel's sources changed since the counters in " + TRAFFIC_PROFILE + " were taken"
    batch = int(b.group(1))
    return total * BATCH / batch, (f"ncu DRAM bytes of the layer-6 launch at batch {batch} from {TRAFFIC_PROFILE}, scaled by "
                                   f"the pixel count to batch {BATCH} (traffic is proportional to pixels; the filter is 1.2 MB)")


def slowest_rank_ms(ms, world, device="cpu"):
    """Max over ranks of a per-rank duration (all-reduce MAX on the default process group)."""
    if world == 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def average_gradients(grads, world):
    """Data-parallel exchange of a training step: every rank ends with the mean of the ranks'
    gradients, i.e. the gradient of the mean loss over the whole job's batch (each rank's loss is
    the mean over its own, equally sized, batch).  One all-reduce on the default process group."""
    if world == 1:
        return grads
    import torch.distributed as dist
    dist.all_reduce(grads, op=dist.ReduceOp.SUM)
    grads /= world
    return grads


def aggregate_images_per_s(world, batch_per_rank, steps, slowest_ms):
    """Whole-job throughput: every rank processes its own batch each step (weak scaling)."""
    return world * batch_per_rank * steps / (slowest_ms * 1e-3)


def oracle_forward_rate(n_images, seed_offset=0):
    """images/s of the fp64 CPU checker's forward pass on n_images of the workload."""
    import numpy as np
    import oracle
    import seeded_inputs as si
    params = si.vgg19_params(H, W, seed=0, bf16_exact=True).astype(np.float64)
    images = si.images(BATCH, H, W, seed=1, bf16_exact=True)[seed_offset:seed_offset + n_images]
    oracle.vgg19_forward(params, images[:1])  # page in code and weights
    t0 = time.perf_counter()
    oracle.vgg19_forward(params, images)
    dt = time.perf_counter() - t0
    return n_images / dt, dt


def run_reference(args):
    """The CPU checker as it stands, timed on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    import seeded_inputs as si
    per_step = 1
    params = si.vgg19_params(H, W, seed=0, bf16_exact=True).astype(np.float64)
    images = si.images(BATCH, H, W, seed=1, bf16_exact=True)
    for i in range(args.warmup):
        oracle.vgg19_forward(params, images[i % BATCH:i % BATCH + per_step])
    t0 = time.perf_counter()
    for i in range(args.steps):
        j = (args.warmup + i) % BATCH
        oracle.vgg19_forward(params, images[j:j + per_step])
    dt = time.perf_counter() - t0
    value = per_step * args.steps / dt
    cores = os.cpu_count()
    sample = f"{per_step} image(s) of the batch of 100 per step, {args.steps} steps, forward only"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "images/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD, "note": "fp64 CPU checker, OpenMP over rows; bounded sample"},
        "cpu_baseline": {"value": value, "unit": "images/s", "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def time_conv_layers(pkg, net, torch, stream, reps=5):
    """Per-layer CUDA-event timing of the convolution kernel on the batch-100 activations
    left in the workspace by a forward pass.  Returns [(layer, ms, flop, path)]."""
    out = []
    desc = pkg.vgg19_describe(net.handle).splitlines()
    scratch = torch.empty(BATCH * 224 * 224 * 64, dtype=torch.bfloat16, device=net.device)
    for l, (s, ci, co) in enumerate(CONV):
        if l == 0:
            continue  # 3 input channels: bound by writing its output (see time_first_layer)
        prev = l - 1
        x = net.saved_tensor(BATCH, pkg.VGG19_MODE_BACKWARD, prev)
        if x.shape[1] != s:  # a pool sits between: input is the pooled tensor
            pool_index = {1: 16, 3: 17, 7: 18, 11: 19, 15: 20}[prev]
            x = net.saved_tensor(BATCH, pkg.VGG19_MODE_BACKWARD, pool_index)
        path = "tcgen05" if "fwd=tcgen05" in desc[1 + l] else "simt"
        with torch.cuda.stream(stream):
            for _ in range(2):
                pkg.vgg19_conv_layer_forward(net.handle, l + 1, x, BATCH, scratch, None, stream)
            evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            for a, b in evs:
                a.record(stream)
                pkg.vgg19_conv_layer_forward(net.handle, l + 1, x, BATCH, scratch, None, stream)
                b.record(stream)
        stream.synchronize()
        time.sleep(KERNEL_GAP_S)
        ms = sum(a.elapsed_time(b) for a, b in evs) / reps
        out.append((l + 1, ms, 2.0 * BATCH * s * s * co * 9 * ci, path))
    return out


def time_conv_layers_backward(pkg, net, torch, stream, images, reps=5):
    """Per-layer CUDA-event timing of the two backward kernels of every convolution at batch 100, on the
    activations a training pass left in the workspace: the input gradient (with the ReLU mask of the layer
    below where the pass applies it there) and the filter + bias gradient (with its finishing kernel).
    The upstream gradient is synthetic: N(0, 1e-3) with half of the entries zero, like a ReLU-masked one.
    Returns [(layer, dgrad_ms or None, wgrad_ms, flop)]."""
    out = []
    n_max = BATCH * 224 * 224 * 64
    dz_all = torch.randn(n_max, dtype=torch.float32, device=net.device).mul_(1e-3)
    dz_all.mul_((torch.rand(n_max, device=net.device) < 0.5).float())
    dz_all = dz_all.to(torch.bfloat16)
    dx_all = torch.empty(n_max, dtype=torch.bfloat16, device=net.device)
    for l, (s, ci, co) in enumerate(CONV):
        if l == 0:
            x, pooled_input = images, False
        else:
            x = net.saved_tensor(BATCH, pkg.VGG19_MODE_BACKWARD, l - 1)
            pooled_input = x.shape[1] != s
            if pooled_input:
                x = net.saved_tensor(BATCH, pkg.VGG19_MODE_BACKWARD, {1: 16, 3: 17, 7: 18, 11: 19, 15: 20}[l - 1])
        dz = dz_all[:BATCH * s * s * co].view(BATCH, s, s, co)
        dx = dx_all[:BATCH * s * s * ci].view(BATCH, s, s, ci)
        dw = torch.empty(co * 9 * ci, dtype=torch.float32, device=net.device)
        db = torch.empty(co, dtype=torch.float32, device=net.device)
        mask = None if pooled_input else x  # after a pool the pass masks in the scatter step instead
        calls = {"wgrad": lambda: pkg.vgg19_conv_layer_backward_ex(net.handle, l + 1, x, dz, BATCH, dw, db, None, None, None, stream)}
        if l > 0:
            calls["dgrad"] = lambda: pkg.vgg19_conv_layer_backward_ex(net.handle, l + 1, None, dz, BATCH, None, None, dx, mask, None, stream)
        ms = {}
        for name, fn in calls.items():
            with torch.cuda.stream(stream):
                for _ in range(2):
                    fn()
                evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
                for a, b in evs:
                    a.record(stream)
                    fn()
                    b.record(stream)
            stream.synchronize()
            time.sleep(KERNEL_GAP_S)
            ms[name] = sum(a.elapsed_time(b) for a, b in evs) / reps
        out.append((l + 1, ms.get("dgrad"), ms["wgrad"], 2.0 * BATCH * s * s * co * 9 * ci))
    return out


def time_dense_layers(pkg, net, torch, stream, reps=5):
    """Per-layer CUDA-event timing of the dense layers at batch 100 through the per-layer entry points: forward
    (GEMM + finishing kernel) and backward (bias gradient, input gradient with its ReLU mask, filter gradient).
    Both stream the layer's weights once and are bound by that: algorithmic bytes = bf16 weights read (forward;
    input gradient) + fp32 filter gradient written.  Returns {name: {...}}."""
    dims = [(7 * 7 * 512, 4096), (4096, 4096), (4096, 1000)]
    out = {}
    for i, (In, Out) in enumerate(dims):
        x = torch.randn(BATCH, In, device=net.device).abs().to(torch.bfloat16)
        dy = (torch.randn(BATCH, Out, device=net.device) * 1e-3).to(torch.bfloat16)
        y = torch.empty(BATCH, Out, dtype=torch.bfloat16, device=net.device)
        yf = torch.empty(BATCH, Out, dtype=torch.float32, device=net.device)
        dx = torch.empty(BATCH, In, dtype=torch.bfloat16, device=net.device)
        dw = torch.empty(Out * In, dtype=torch.float32, device=net.device)
        db = torch.empty(Out, dtype=torch.float32, device=net.device)
        calls = {"fwd": lambda: pkg.vgg19_dense_layer_forward(net.handle, i + 1, x, BATCH, y if i < 2 else None, yf if i == 2 else None, stream),
                 "bwd": lambda: pkg.vgg19_dense_layer_backward(net.handle, i + 1, x, dy, BATCH, dw, db, dx, x if i > 0 else None, stream)}
        row = {}
        for name, fn in calls.items():
            with torch.cuda.stream(stream):
                for _ in range(2):
                    fn()
                evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
                for a, b in evs:
                    a.record(stream)
                    fn()
                    b.record(stream)
            stream.synchronize()
            time.sleep(KERNEL_GAP_S)
            row[name] = sum(a.elapsed_time(b) for a, b in evs) / reps
        w = In * Out
        out[f"dense{i + 1}"] = {"fwd_ms": row["fwd"], "fwd_bytes": 2 * w + 2 * BATCH * (In + Out),
                                "bwd_ms": row["bwd"], "bwd_bytes": 2 * w + 4 * w + 2 * BATCH * (2 * In + 2 * Out)}
        del x, dy, y, yf, dx, dw, db
    return out


def forward_roofline_ms(pk):
    """Kernel-by-kernel roofline of the forward pass at batch 100: sum over its steps of
    max(flop / tensor peak, bytes / copy bandwidth), with each activation written once and read once
    (pooled where the pool is fused), the image read once, weights read once."""
    tf, bw = pk["bf16_tflops"] * 1e12, pk["hbm_gbs"] * 1e9
    pool_after = {1, 3, 7, 11, 15}
    total = 0.0
    for l, (s, ci, co) in enumerate(CONV):
        flop = 2.0 * BATCH * s * s * co * 9 * ci
        out_px = BATCH * s * s // (4 if l in pool_after else 1)
        byts = 2.0 * (BATCH * s * s * ci + out_px * co + 9 * ci * co)
        total += max(flop / tf, byts / bw)
    for i, o in ((25088, 4096), (4096, 4096), (4096, 1000)):
        total += max(2.0 * BATCH * i * o / tf, 2.0 * (i * o + BATCH * (i + o)) / bw)
    return total * 1e3


def time_first_layer(pkg, net, torch, stream, x, reps=5):
    """conv1_1 (3 -> 64 channels), the pass's largest memory-bound kernel: CUDA-event time of the layer
    (channel-padding copy + convolution) and the algorithmic bytes it has to move: the 3-channel image in,
    the 64-channel activation out."""
    y = torch.empty(BATCH, H, W, 64, dtype=torch.bfloat16, device=net.device)
    with torch.cuda.stream(stream):
        for _ in range(2):
            pkg.vgg19_conv_layer_forward(net.handle, 1, x, BATCH, y, None, stream)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b in evs:
            a.record(stream)
            pkg.vgg19_conv_layer_forward(net.handle, 1, x, BATCH, y, None, stream)
            b.record(stream)
    stream.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in evs) / reps
    return ms, BATCH * H * W * (3 + 64) * 2


def run_native(args):
    import numpy as np
    import torch
    import seeded_inputs as si
    import paper_1810_09868_b200 as pkg

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
        if rank == 0:
            print(f"bench: {world} ranks, one GPU each, NCCL communicator of size {dist.get_world_size()}", file=sys.stderr)

    params = si.vgg19_params(H, W, seed=0, bf16_exact=True)
    images = si.images(BATCH, H, W, seed=1, bf16_exact=True)
    labels = si.labels(BATCH, seed=2)
    # the training-step workspace (backward pass + gradient buffer) also covers the forward pass and its
    # two host-staging slots
    net = pkg.Net(H, W, BATCH, pkg.VGG19_BF16, params=params, mode=pkg.VGG19_MODE_TRAIN, device=f"cuda:{local}")
    assert net.workspace.numel() >= (pkg.vgg19_workspace_bytes(net.handle, BATCH, pkg.VGG19_MODE_FORWARD)
                                     + pkg.vgg19_io_bytes(net.handle, BATCH, pkg.VGG19_MODE_FORWARD))
    x = torch.from_numpy(images).to(dev).to(torch.bfloat16)
    y = torch.from_numpy(labels).to(dev)
    logits = torch.empty(BATCH, 1000, dtype=torch.float32, device=dev)
    grads = torch.empty(net.n_params, dtype=torch.float32, device=dev)
    loss = torch.empty(1, dtype=torch.float32, device=dev)
    stream = torch.cuda.Stream(device=dev)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def max_over_ranks(ms):
        return slowest_rank_ms(ms, world, dev)

    def timed(fn, steps, warmup):
        with torch.cuda.stream(stream):
            for _ in range(warmup):
                fn()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            a.record(stream)
            for _ in range(steps):
                fn()
            b.record(stream)
        barrier()
        return max_over_ranks(a.elapsed_time(b))

    fwd = lambda: pkg.vgg19_forward(net.handle, x, BATCH, logits, None, stream)
    bwd = lambda: pkg.vgg19_backward(net.handle, x, y, BATCH, grads, loss, None, stream)

    side = torch.cuda.Stream(device=dev)
    dense_off, _ = pkg.vgg19_param_info(net.handle, 32)
    dense_ready = torch.cuda.Event()
    dense_ready.record(stream)  # creates the handle the library records into

    def train():
        if world == 1:
            # one GPU: forward, loss, backward and the update of every parameter copy as ONE recorded graph
            pkg.vgg19_train_step(net.handle, x, y, BATCH, TRAIN_LR, loss, stream)
            return
        # several GPUs: the backward pass signals `dense_ready` once the dense layers' gradients (86 % of
        # the buffer) are final; their all-reduce runs on a side stream beside the convolution layers'
        # backward pass, the convolution gradients are exchanged when the pass ends, then one SGD step
        pkg.vgg19_backward(net.handle, x, y, BATCH, grads, loss, None, stream)
        with torch.cuda.stream(side):
            side.wait_event(dense_ready)
            average_gradients(grads[dense_off:], world)
        average_gradients(grads[:dense_off], world)
        stream.wait_stream(side)
        pkg.vgg19_sgd_step(net.handle, grads, TRAIN_LR, stream)

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.6)  # nvidia-smi needs a moment before its first sample
    t_begin = time.time()
    fwd_ms = timed(fwd, args.steps, args.warmup)
    net.sync_status(stream)
    t_end_fwd = time.time()
    # Per-kernel timings come next, on a GPU that has run for a few tens of milliseconds only: they are
    # compared with burst peaks (a best-of-10 GEMM and copy on an idle GPU), and the seconds of sustained
    # load further down pull the SM clock to the power cap's level.  Rank 0 only; the others wait at the
    # next barrier.
    layers = bwd_layers = dense_layers = None
    t_k0 = time.time()
    if rank == 0:
        with torch.cuda.stream(stream):
            bwd()  # leaves the batch-100 activations of every layer in the workspace
        stream.synchronize()
        time.sleep(0.3)
        layers = time_conv_layers(pkg, net, torch, stream)
        first_ms, first_bytes = time_first_layer(pkg, net, torch, stream, x)
        bwd_layers = time_conv_layers_backward(pkg, net, torch, stream, x)
        dense_layers = time_dense_layers(pkg, net, torch, stream)
        t_k1 = time.time()
        time.sleep(1.0)  # let the power budget recover before the next timed region
    bwd_steps = max(3, args.steps // 2)
    t_begin_bwd = time.time()
    bwd_ms = timed(bwd, bwd_steps, max(3, args.warmup))
    t_end = time.time()
    net.sync_status(stream)
    # sustained: back-to-back forward passes for about args.sustained_s seconds (the power cap settles the
    # SM clock within the first second), timed as one region
    sustained_steps = max(args.steps, int(args.sustained_s * 1e3 / (fwd_ms / args.steps)))
    t_sus0 = time.time()
    sustained_ms = timed(fwd, sustained_steps, 0)
    t_sus1 = time.time()
    net.sync_status(stream)
    # the clock record of the headline number: the samples inside the forward passes' timed region
    clocks = sampler.stop(t_begin, t_end_fwd, extra_window=(t_sus0, t_sus1), kernel_window=(t_k0, t_k1)) if sampler else None
    sustained_clocks = clocks.pop("extra", None) if clocks else None
    kernel_clocks = clocks.pop("kernels", None) if clocks else None

    # training step last: it moves the weights (by a learning rate small enough to keep them sane)
    if world > 1:
        pkg.vgg19_set_dense_grads_event(net.handle, dense_ready)
    train_steps = max(3, args.steps // 2)
    train_ms = timed(train, train_steps, 3)
    net.sync_status(stream)

    # end to end: pinned host images in, logits out, through the host-buffer entry point
    x_host = torch.from_numpy(images).to(torch.bfloat16).pin_memory()
    logits_host = torch.empty(BATCH, 1000, dtype=torch.float32).pin_memory()
    # (every step uploads its own 30 MB of images and downloads its logits; the upload of step k+1
    # runs on the library's copy stream while step k computes)
    for _ in range(max(3, args.warmup)):
        pkg.vgg19_forward_host_async(net.handle, x_host, BATCH, logits_host, None, stream)
    net.sync_status(stream)
    barrier()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        pkg.vgg19_forward_host_async(net.handle, x_host, BATCH, logits_host, None, stream)
    net.sync_status(stream)
    e2e_ms = max_over_ranks(1e3 * (time.perf_counter() - t0))
    barrier()
    # the blocking call, one batch at a time (upload, pass, download, wait), for comparison
    t0 = time.perf_counter()
    for _ in range(args.steps):
        pkg.vgg19_forward_host(net.handle, x_host, BATCH, logits_host, None, stream)
    e2e_blocking_ms = max_over_ranks(1e3 * (time.perf_counter() - t0))
    barrier()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    pk = peaks()
    # roofline of the dominant kernel: the convolution layers after the first (timed above)
    # dominant kernel: conv3x3_pair_tc_kernel<256>, the 12 launches of layers 5..16 (60 % of the pass)
    dom = [t for t in layers if t[0] >= 5]
    conv_ms = sum(ms for _, ms, _, _ in dom)
    conv_flop = sum(f for _, _, f, _ in dom)
    achieved = conv_flop / (conv_ms * 1e-3) / 1e12
    all_ms = sum(ms for _, ms, _, _ in layers)
    all_flop = sum(f for _, _, f, _ in layers)
    peak = pk["bf16_tflops"]
    per_layer = {f"conv{l}": {"ms": round(ms, 4), "tflops": round(f / (ms * 1e-3) / 1e12, 1), "path": path}
                 for l, ms, f, path in layers}
    traffic, traffic_note = dominant_kernel_traffic()
    traffic_per_launch = None if traffic is None else traffic  # the layer-6 launch; one of the 12 timed here
    # backward kernels per layer, and every tensor-bound kernel below 60 % of the bf16 peak
    per_layer_bwd, below = {}, []
    for l, dg, wg, f in bwd_layers:
        row = {"wgrad_ms": round(wg, 4)}
        if l == 1:
            # filter gradient of the 3-channel layer: bound by reading dz (642 MB) and the image
            byts = BATCH * H * W * (64 + 3) * 2
            row["wgrad_gbs"] = round(byts / (wg * 1e-3) / 1e9, 1)
            row["wgrad_frac_of_hbm"] = round(byts / (wg * 1e-3) / 1e9 / pk["hbm_gbs"], 3)
        else:
            row["wgrad_tflops"] = round(f / (wg * 1e-3) / 1e12, 1)
            row["wgrad_frac"] = round(f / (wg * 1e-3) / 1e12 / peak, 3)
            row["dgrad_ms"] = round(dg, 4)
            row["dgrad_tflops"] = round(f / (dg * 1e-3) / 1e12, 1)
            row["dgrad_frac"] = round(f / (dg * 1e-3) / 1e12 / peak, 3)
            # an input gradient reads dz and the ReLU mask of the layer below and writes dx: where those bytes at the
            # measured copy bandwidth take longer than the FLOPs at the tensor peak, that is the kernel's roofline
            s_, ci, co = CONV[l - 1]
            hbm_ms = BATCH * s_ * s_ * (co + 2 * ci) * 2 / (pk["hbm_gbs"] * 1e9) * 1e3
            if hbm_ms > f / (peak * 1e12) * 1e3:
                row["dgrad_bound"] = "hbm"
                row["dgrad_hbm_floor_ms"] = round(hbm_ms, 4)
                row["dgrad_frac_of_hbm"] = round(hbm_ms / dg, 3)
            for kind in ("wgrad", "dgrad"):
                if row[kind + "_frac"] < 0.6:
                    hb = f" (hbm-bound: {row['dgrad_frac_of_hbm']:.2f} of its byte floor)" if kind == "dgrad" and "dgrad_bound" in row else ""
                    below.append(f"conv{l} {kind} {row[kind + '_frac']:.2f}{hb}")
        per_layer_bwd[f"conv{l}"] = row
    for l, ms, f, path in layers:
        if f / (ms * 1e-3) / 1e12 / peak < 0.6:
            below.append(f"conv{l} fwd {f / (ms * 1e-3) / 1e12 / peak:.2f}")
    # dense layers: bound by streaming their weights (and, backward, writing the fp32 filter gradient)
    per_dense = {}
    for name, d in dense_layers.items():
        per_dense[name] = {"fwd_ms": round(d["fwd_ms"], 4), "fwd_gbs": round(d["fwd_bytes"] / (d["fwd_ms"] * 1e-3) / 1e9, 1),
                           "fwd_frac_of_hbm": round(d["fwd_bytes"] / (d["fwd_ms"] * 1e-3) / 1e9 / pk["hbm_gbs"], 3),
                           "bwd_ms": round(d["bwd_ms"], 4), "bwd_gbs": round(d["bwd_bytes"] / (d["bwd_ms"] * 1e-3) / 1e9, 1),
                           "bwd_frac_of_hbm": round(d["bwd_bytes"] / (d["bwd_ms"] * 1e-3) / 1e9 / pk["hbm_gbs"], 3)}
    bwd_conv_ms = sum((dg or 0.0) + wg for _, dg, wg, _ in bwd_layers)
    bwd_conv_flop = sum(f * (2 if l > 1 else 0) for l, _, _, f in bwd_layers)
    roof_ms = forward_roofline_ms(pk)

    n_fwd = pkg.vgg19_launch_count(net.handle, pkg.VGG19_MODE_FORWARD)
    cpu_rate, cpu_dt = oracle_forward_rate(args.cpu_images)
    value = aggregate_images_per_s(world, BATCH, args.steps, fwd_ms)
    fwd_tflops = value * FWD_FLOP_PER_IMAGE / 1e12 / world
    out = {
        "metric": METRIC, "value": value, "unit": "images/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": fwd_ms / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": BATCH, "image": [H, W, 3],
                   "l2": "no explicit flush: each step writes and re-reads 2.1 GB of activations, 16x the 126 MB L2",
                   "weights": "He-normal seed 0, biases 0", "graph": "one CUDA graph per pass"},
        "clocks": clocks,
        "e2e": {"value": world * BATCH * args.steps / (e2e_ms * 1e-3), "unit": "images/s",
                "h2d_bytes_per_step": x_host.numel() * 2, "d2h_bytes_per_step": logits_host.numel() * 4,
                "api": "vgg19_forward_host_async (uploads overlap the previous batch's pass), wall clock over all steps",
                "blocking_call_value": world * BATCH * args.steps / (e2e_blocking_ms * 1e-3)},
        "gpu_launches": n_fwd * args.steps,
        "fwd_tflops_per_gpu": fwd_tflops,
        "fwd_frac_of_bf16_peak": fwd_tflops / peak,
        "fwd_frac_of_roofline": roof_ms / (fwd_ms / args.steps),
        "fwd_roofline_ms": roof_ms,
        "sustained": {"value": aggregate_images_per_s(world, BATCH, sustained_steps, sustained_ms), "unit": "images/s",
                      "steps": sustained_steps, "seconds": sustained_ms * 1e-3, "ms_per_step": sustained_ms / sustained_steps,
                      "tflops_per_gpu": BATCH * sustained_steps / (sustained_ms * 1e-3) * FWD_FLOP_PER_IMAGE / 1e12,
                      "frac_of_sustained_bf16_peak": BATCH * sustained_steps / (sustained_ms * 1e-3) * FWD_FLOP_PER_IMAGE / 1e12
                                                     / pk["bf16_tflops_sustained"],
                      "clocks": sustained_clocks},
        "fwd_bwd": {"value": world * BATCH * bwd_steps / (bwd_ms * 1e-3), "unit": "images/s", "steps": bwd_steps,
                    "ms_per_step": bwd_ms / bwd_steps,
                    "launches_per_step": pkg.vgg19_launch_count(net.handle, pkg.VGG19_MODE_BACKWARD)},
        "train_step": {"value": world * BATCH * train_steps / (train_ms * 1e-3), "unit": "images/s", "steps": train_steps,
                       "ms_per_step": train_ms / train_steps, "lr": TRAIN_LR,
                       "what": ("vgg19_train_step: forward + backward + SGD update of the fp32 master, bf16 and filter "
                                "copies as one CUDA graph" if world == 1 else
                                "vgg19_backward + NCCL all-reduce of the dense gradients (494 MB) on a side stream from "
                                "the point the pass signals them final, of the convolution gradients (80 MB) at its "
                                "end + vgg19_sgd_step"),
                       "launches_per_step": pkg.vgg19_launch_count(net.handle, pkg.VGG19_MODE_TRAIN) if world == 1 else None},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                     "frac": achieved / peak, "traffic": traffic_per_launch,
                     "kernel": "conv3x3_pair_tc_kernel<256>: 3x3 convolution forward as a tcgen05 cta_group::2 implicit "
                               "GEMM on CTA pairs, layers 5..16 (12 launches per pass), algorithmic flops / summed launch time",
                     "traffic_note": traffic_note + "; algorithmic bytes of that launch: 160.6 MB in + 160.6 MB out + 1.2 MB "
                                     "filter (the output is partly still in L2 when the launch ends)",
                     "peak_source": f"{pk['source']} burst bf16 GEMM (kernel timed alone per layer)",
                     "all_conv_layers_2_16": {"tflops": all_flop / (all_ms * 1e-3) / 1e12,
                                              "frac": all_flop / (all_ms * 1e-3) / 1e12 / peak},
                     "per_layer": per_layer,
                     "per_layer_bwd": per_layer_bwd,
                     "per_dense_layer": per_dense,
                     "per_kernel_clocks": kernel_clocks,
                     "bwd_conv_kernels": {"ms": bwd_conv_ms, "tflops": bwd_conv_flop / (bwd_conv_ms * 1e-3) / 1e12,
                                          "note": "input- and filter-gradient kernels of layers 1..16, each timed alone"},
                     "below_60pct_of_bf16_peak": below,
                     "hbm_bound_not_listed_above": "conv1 fwd and wgrad (3 input channels) and the dense layers (per_dense_layer) at batch "
                                                   "100 are bound by HBM, see hbm_bound and per_layer_bwd.conv1"},
        "hbm_bound": {"kernel": "conv1_1 forward (pad_to8_kernel + conv3x3_c8_tc_kernel): 3-channel image in, 64-channel activation out",
                      "ms": round(first_ms, 4), "achieved": first_bytes / (first_ms * 1e-3) / 1e9, "peak": pk["hbm_gbs"],
                      "unit": "GB/s", "frac": first_bytes / (first_ms * 1e-3) / 1e9 / pk["hbm_gbs"],
                      "peak_source": f"{pk['source']} copy bandwidth"},
        "cpu_baseline": {"value": cpu_rate, "unit": "images/s", "cores": os.cpu_count(), "kind": "oracle",
                         "sample": f"forward of {args.cpu_images} of the 100 images, {cpu_dt:.1f} s"},
        "context": {"paper_tpuv2_core_s_per_batch100": 0.23, "paper_xeon_4114_flux_cpu_s_per_batch100": 52.4},
    }
    print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(args):
    """`python bench.py --gpus N` without a launcher: start N ranks of this script, one per GPU, through
    torch.distributed.run on 127.0.0.1 and hand their exit status back."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    env = dict(os.environ)
    if args.backend == "nccl":
        # the communicator's size and transport show in NCCL's own start-up lines (stderr)
        env.setdefault("NCCL_DEBUG", "INFO")
        env.setdefault("NCCL_DEBUG_SUBSYS", "INIT")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd, env=env)


def run_dry(args):
    """The multi-rank plumbing of run_native without a GPU: rendezvous, barrier, max over ranks of a
    per-rank duration, gradient averaging, whole-job aggregation.  Each rank pretends its pass took
    (10 + rank) ms per step and that its gradient is the constant rank + 1."""
    import torch
    import torch.distributed as dist
    if args.backend != "gloo":
        raise SystemExit("--dry runs on CPU ranks: use --backend gloo")
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
        dist.barrier()
    ms = slowest_rank_ms((10.0 + rank) * args.steps, world)
    g = average_gradients(torch.full((8,), float(rank + 1)), world)
    if rank == 0:
        print(json.dumps({"metric": METRIC, "dry": True, "n_gpus": world, "steps": args.steps,
                          "value": aggregate_images_per_s(world, BATCH, args.steps, ms), "unit": "images/s",
                          "ms_per_step": ms / args.steps, "mean_gradient": float(g[0]), "scaling": "weak"}))
    if world > 1:
        dist.destroy_process_group()


def run_profile_layer(args):
    """A few launches of one convolution layer on a small batch, for `ncu -k ...` captures
    (prints nothing the driver parses)."""
    import torch
    import seeded_inputs as si
    import paper_1810_09868_b200 as pkg
    L, B = args.profile_layer, args.profile_batch
    s, ci, co = CONV[L - 1]
    if args.profile_kind == "split":
        # the fp32 configuration's tensor-core path: fp32 tensors in and out, split-fp16 kernel between
        params = si.vgg19_params(H, W, seed=0)
        net = pkg.Net(H, W, B, pkg.VGG19_FP32, params=params, flags=pkg.VGG19_FLAG_SPLIT_F16, mode=pkg.VGG19_MODE_FORWARD)
        x = torch.from_numpy(si.normal(B * s * s * ci, seed=100 + L, take_abs=True).reshape(B, s, s, ci)).cuda().float()
        y = torch.empty(B, s, s, co, dtype=torch.float32, device="cuda")
        stream = torch.cuda.Stream()
        for _ in range(3):
            pkg.vgg19_conv_layer_forward(net.handle, L, x, B, y, None, stream)
        net.sync_status(stream)
        print(f"profiled conv layer {L} (split-fp16), batch {B}: {s}x{s}, {ci}->{co}")
        return
    params = si.vgg19_params(H, W, seed=0, bf16_exact=True)
    net = pkg.Net(H, W, B, pkg.VGG19_BF16, params=params)
    x = torch.from_numpy(si.normal(B * s * s * ci, seed=100 + L, take_abs=True, bf16_exact=True)
                         .reshape(B, s, s, ci)).cuda().to(torch.bfloat16)
    y = torch.empty(B, s, s, co, dtype=torch.bfloat16, device="cuda")
    stream = torch.cuda.Stream()
    if args.profile_kind == "fwd":
        for _ in range(3):
            pkg.vgg19_conv_layer_forward(net.handle, L, x, B, y, None, stream)
    else:
        dz = torch.from_numpy(si.normal(B * s * s * co, seed=200 + L, stddev=1e-3, bf16_exact=True)
                              .reshape(B, s, s, co)).cuda().to(torch.bfloat16)
        dw = torch.empty(co, 3, 3, ci, dtype=torch.float32, device="cuda")
        db = torch.empty(co, dtype=torch.float32, device="cuda")
        dx = None if L == 1 else torch.empty(B, s, s, ci, dtype=torch.bfloat16, device="cuda")
        for _ in range(3):
            pkg.vgg19_conv_layer_backward(net.handle, L, x, dz, B, dw, db, dx, stream)
    net.sync_status(stream)
    print(f"profiled conv layer {L} ({args.profile_kind}), batch {B}: {s}x{s}, {ci}->{co}")


def run_profile_pass(args):
    """Three forward passes, then three forward+backward passes at the benchmark's batch, and nothing else:
    the launch list of `ncu --metrics gpu__time_duration.sum` on this is the per-kernel share of a pass
    (prints nothing the driver parses)."""
    import torch
    import seeded_inputs as si
    import paper_1810_09868_b200 as pkg
    params = si.vgg19_params(H, W, seed=0, bf16_exact=True)
    net = pkg.Net(H, W, BATCH, pkg.VGG19_BF16, params=params)
    x = torch.from_numpy(si.images(BATCH, H, W, seed=1, bf16_exact=True)).cuda().to(torch.bfloat16)
    y = torch.from_numpy(si.labels(BATCH, seed=2)).cuda()
    logits = torch.empty(BATCH, 1000, dtype=torch.float32, device="cuda")
    grads = torch.empty(net.n_params, dtype=torch.float32, device="cuda")
    loss = torch.empty(1, dtype=torch.float32, device="cuda")
    stream = torch.cuda.Stream()
    for _ in range(3):
        pkg.vgg19_forward(net.handle, x, BATCH, logits, None, stream)
    for _ in range(3):
        pkg.vgg19_backward(net.handle, x, y, BATCH, grads, loss, None, stream)
    net.sync_status(stream)
    print(f"profiled 3 forward passes ({pkg.vgg19_launch_count(net.handle, pkg.VGG19_MODE_FORWARD)} kernels each) and 3 "
          f"forward+backward passes ({pkg.vgg19_launch_count(net.handle, pkg.VGG19_MODE_BACKWARD)} kernels each)")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--cpu-images", type=int, default=24, help="images the CPU checker is timed on")
    ap.add_argument("--sustained-s", type=float, default=2.5, help="seconds of back-to-back passes for the sustained figure")
    ap.add_argument("--backend", default="nccl", choices=["nccl", "gloo"])
    ap.add_argument("--dry", action="store_true", help="multi-rank plumbing only, on CPU ranks (needs --backend gloo)")
    ap.add_argument("--profile-layer", type=int, default=0, help="run only this conv layer (1..16) a few times and exit")
    ap.add_argument("--profile-pass", action="store_true", help="run three forward and three forward+backward passes and exit")
    ap.add_argument("--profile-batch", type=int, default=16)
    ap.add_argument("--profile-kind", default="fwd", choices=["fwd", "bwd", "split"])
    args = ap.parse_args()
    if args.profile_layer:
        run_profile_layer(args)
        return
    if args.profile_pass:
        run_profile_pass(args)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args))
    elif args.dry:
        run_dry(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()

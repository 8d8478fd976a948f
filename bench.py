#!/usr/bin/env python3
"""Benchmark of the DDG training step: images/sec of one DDG iteration (ResNet-110, K=4, batch 128, bf16 storage)
on synthetic CIFAR-shaped data, one B200 per process.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--net resnet110] [--modules 4]

N > 1 (under torchrun) runs N independent replicas (the method does not shard across GPUs here): `value` is the sum
over replicas, timed as the max over ranks.  `--impl reference` times the CPU oracle on a bounded sample of the same
workload on the host cores.  One JSON line is printed by rank 0.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "DDG train images/sec (ResNet-110, K=4, 1 B200)"


def parse():
    p = argparse.ArgumentParser()
    p.add_argument("--gpus", type=int, default=1)
    p.add_argument("--steps", type=int, default=200)
    p.add_argument("--warmup", type=int, default=20)
    p.add_argument("--impl", default="ours", choices=["ours", "reference"])
    p.add_argument("--net", default="resnet110", choices=["resnet110", "resnet56", "resnet8", "mlp"])
    p.add_argument("--modules", type=int, default=0, help="K; 0 = the configuration's own split")
    p.add_argument("--batch", type=int, default=0)
    p.add_argument("--no-graph", action="store_true")
    p.add_argument("--cpu-batch", type=int, default=8, help="batch of the bounded CPU-oracle sample")
    p.add_argument("--cpu-steps", type=int, default=0, help="timed oracle iterations (0 = 20 beside the GPU arm; "
                   "min(--steps, 100) for --impl reference)")
    p.add_argument("--skip-cpu", action="store_true")
    p.add_argument("--skip-k1", action="store_true", help="leave out the K = 1 arm")
    p.add_argument("--fuse-bn-apply", type=int, default=0, help="ddg_cfg.fuse_bn_apply (A/B runs)")
    p.add_argument("--bn-fold", type=int, default=0, help="ddg_cfg.bn_fold (A/B runs)")
    return p.parse_args()


def workload(args):
    from paper_1804_10574_b200 import nets
    cfg = dict(nets.config(args.net))
    if args.modules:
        cfg["split_after"] = nets.split_even_blocks(cfg["layers"], args.modules) if args.net.startswith("resnet") \
            else cfg["split_after"]
    if args.batch:
        cfg["batch"] = args.batch
    return cfg


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "20"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass
        sm = [float(r[0]) for r in self.rows if len(r) >= 7 and r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in self.rows if len(r) >= 7 and r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(len(r) >= 7 and r[3 + i] == "Active" for r in self.rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": reasons, "samples": len(sm)}


def time_oracle(cfg, batch, n_steps):
    """The CPU oracle as it stands, on a bounded sample of the workload: same net and split, smaller batch."""
    from oracle import ddg_oracle as orc
    from paper_1804_10574_b200 import synth
    K = len(cfg["split_after"]) + 1
    o = cfg["opt"]
    ref = orc.Oracle(cfg["layers"], cfg["split_after"], batch, cfg["in_shape"], cfg["num_classes"], lr=o["lr"],
                     momentum=o["momentum"], weight_decay=o["weight_decay"],
                     flags=orc.ROUND_BF16 if cfg["precision"] == "bf16" else orc.ROUND_FP32)
    ref.set_weights(synth.init_weights(cfg["layers"]).astype(np.float64))
    data = [synth.batch(t, batch, cfg["in_shape"], cfg["num_classes"]) for t in range(K - 1 + n_steps)]
    for t in range(K - 1):                      # fill the pipeline: untimed
        ref.step(*data[t])
    t0 = time.perf_counter()
    for t in range(K - 1, K - 1 + n_steps):
        ref.step(*data[t])
    dt = time.perf_counter() - t0
    ref.close()
    cores = len(os.sched_getaffinity(0))
    threads = int(os.environ.get("OMP_NUM_THREADS", cores))
    return {"value": batch * n_steps / dt, "unit": "images/s", "cores": min(cores, threads), "kind": "oracle",
            "sample": "%d full DDG iterations of the same network and split at batch %d (of %d), fp64, after K-1 "
                      "untimed pipeline-fill iterations" % (n_steps, batch, cfg["batch"]), "seconds": dt}


def _time_back_to_back(torch, launches, stream, reps=5):
    """Average device time of one launch when `launches` (callables on distinct buffers, together larger than L2) run
    back to back, as the kernels of a training step do.  The sequence is recorded once into a CUDA graph on a side
    stream and replayed (the step replays graphs too): enqueueing one launch at a time from Python takes longer than
    a launch runs, which would time the interpreter instead of the kernels.  CUDA events around each replay."""
    side = torch.cuda.Stream()
    for fn in launches[:3]:
        fn(stream.cuda_stream)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=side):
        for fn in launches:
            fn(side.cuda_stream)
    for _ in range(2):
        graph.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        graph.replay()
        e1.record(stream)
        e1.synchronize()
        ts.append(e0.elapsed_time(e1) * 1e-3 / len(launches))
    return float(np.median(ts))


def ncu_counters():
    """Figures copied from the ncu summaries under profiles/ (DRAM bytes of the dominant kernel, its share of the
    launch list), kept in profiles/roofline_counters.json beside the summaries they come from.  Each entry names the
    source file of its kernel with the hash that file had when the counters were taken: a kernel that has changed
    since has no valid counters, and its figure is reported as null."""
    import hashlib
    try:
        doc = json.load(open(os.path.join(ROOT, "profiles", "roofline_counters.json")))
    except Exception:
        return {}
    out = {}
    for name, ent in doc.items():
        try:
            src = open(os.path.join(ROOT, ent["kernel_source"]), "rb").read()
            ent = dict(ent, valid=hashlib.sha256(src).hexdigest() == ent["kernel_source_sha256"])
        except Exception:
            ent = dict(ent, valid=False)
        out[name] = ent
    return out


def dominant_kernel_roofline(torch, binding, cfg, peaks, K):
    """The kernel with the largest share of the ncu launch list of this workload is the tensor-core convolution on the
    16-channel 32x32 maps, conv3x3_tc_kernel<16> (profiles/ddg_step_resnet110_k4_b128_bf16_launch_list.md).  It is
    timed here at the step's shape and launch configuration, with its pre-arranged filter image, as a sequence of
    launches on distinct tensors (more than L2 in total), replayed as one CUDA graph between two CUDA events.  The other
    convolution widths and the batch-norm backward pass are timed the same way and listed beside it."""
    B = cfg["batch"]
    bf = torch.bfloat16
    s = torch.cuda.current_stream()
    hbm = peaks.get("hbm_gbs", 6650.0)
    tflops = peaks.get("bf16_tflops", 1590.0)
    src = "measured" if "hbm_gbs" in peaks else "fallback"

    def conv_case(Hh, Cc, B=B, form="plain"):
        """form: "plain" = the convolution alone; "stats" = with the batch-norm statistics epilogue, sums folded by the
        CTA that finishes last (what the step launches while module streams share the GPU), timed with the launch plan
        of a kernel that has the GPU to itself, as a kernel timed alone does; "stats_shared" = the same with the plan the
        K > 1 step gives it (fewer CTAs, so that the other modules' kernels fit beside it: slower alone by design);
        "partials" = the epilogue leaves per-CTA partial sums for the element-wise pass (what a single stream launches)."""
        per = 2 * B * Hh * Hh * Cc * 2                       # bytes of input + output of one launch
        n = max(8, int(400e6 // per) + 1) if B <= 1024 else max(2, int(400e6 // per) + 1)
        xs = [torch.randn(B, Hh, Hh, Cc, device="cuda").to(bf) for _ in range(n)]
        ys = [torch.empty_like(xs[0]) for _ in range(n)]
        w = (torch.randn(Cc, Cc, 3, 3, device="cuda") * (2.0 / (9 * Cc)) ** 0.5).to(bf)
        pk = torch.empty(binding.conv3x3_packed_bytes(B, Hh, Hh, Cc), dtype=torch.uint8, device="cuda")
        binding.conv3x3_pack(w, pk, Cc)
        m, iv = torch.empty(Cc, device="cuda"), torch.empty(Cc, device="cuda")
        scr = torch.zeros(binding.conv3x3_fused_scratch_elems(B, Hh, Hh, Cc), device="cuda")
        if form == "stats":
            fns = [(lambda st, i=i: binding.conv3x3_fwd_stats_prepared(xs[i], w, pk, ys[i], m, iv, scr, B, Hh, Hh, Cc, st)) for i in range(n)]
        elif form == "stats_shared":
            # the launch plan of a step with several module streams (fewer CTAs, at least two tiles per pipeline)
            fns = [(lambda st, i=i: binding.conv3x3_fwd_stats_shared(xs[i], w, pk, ys[i], m, iv, scr, B, Hh, Hh, Cc, st)) for i in range(n)]
        elif form == "partials":
            fns = [(lambda st, i=i: binding.conv3x3_fwd_partials(xs[i], w, pk, ys[i], scr, B, Hh, Hh, Cc, st)) for i in range(n)]
        else:
            fns = [(lambda st, i=i: binding.conv3x3_packed(0, xs[i], w, pk, ys[i], B, Hh, Hh, Cc, st)) for i in range(n)]
        dt = _time_back_to_back(torch, fns, s)
        return dt, per + w.numel() * 2, 2.0 * 9 * Cc * Cc * B * Hh * Hh, n

    # the dominant kernel in the form the benchmarked step launches it: with its batch-norm statistics epilogue
    step_form = "stats" if K > 1 else "partials"
    dt, alg, flops, n = conv_case(32, 16, form=step_form)
    # DRAM traffic per launch from the ncu capture at batch 4096 (read + written; part of the output is still in L2
    # when the kernel ends); traffic grows with the pixels processed, so it is scaled by batch.  null when the kernel's
    # source has changed since the capture.
    cnt = ncu_counters()
    c16 = cnt.get("conv3x3_tc_kernel<16> fwd 32x32")
    traffic = None
    if c16 and c16["valid"]:
        traffic = (c16["dram_bytes_read"] + c16["dram_bytes_write"]) * B / float(c16["batch"])
    share = cnt.get("launch_list resnet110 K=4 B=128", {})
    roof = {"kernel": "conv3x3_tc_kernel<16> (tensor-core 3x3 convolution, forward, with the batch-norm statistics "
                      "epilogue as the step launches it: %s; timed alone, with the grid of a kernel that has the GPU to "
                      "itself) C=16 32x32 B=%d"
                      % ("sums folded by the last CTA" if K > 1 else "per-CTA partial sums left to the element-wise pass", B),
            "bound": "hbm",
            "achieved": alg / dt / 1e9, "peak": hbm, "unit": "GB/s", "frac": alg / dt / 1e9 / hbm, "traffic": traffic,
            "launch_us": dt * 1e6, "peak_source": src,
            "ncu_share_of_step": share.get("conv3x3_tc_kernel<16>") if share.get("valid") else None, "launches_timed": n,
            "tflops": flops / dt / 1e12, "tensor_frac": flops / dt / 1e12 / tflops}
    others = []
    for form in ("plain", "stats", "stats_shared", "partials"):
        if form == step_form:
            continue
        dtc, nbytes, fl, _ = conv_case(32, 16, form=form)
        others.append({"kernel": "conv3x3_tc_kernel<16> fwd 32x32 B=%d, %s" % (B, {"plain": "without the statistics epilogue",
                       "stats": "statistics folded by the last CTA",
                       "stats_shared": "statistics folded by the last CTA, launch plan of the K > 1 step (fewer CTAs, leaves "
                                       "SMs to the other module streams)",
                       "partials": "partial sums left to the element-wise pass"}[form]),
                       "launch_us": dtc * 1e6, "hbm_gbs": nbytes / dtc / 1e9, "hbm_frac": nbytes / dtc / 1e9 / hbm})
    for (Hh, Cc) in ((16, 32), (8, 64)):
        dtc, nbytes, fl, _ = conv_case(Hh, Cc)
        others.append({"kernel": "conv3x3_tc_kernel<%d> fwd %dx%d B=%d" % (Cc, Hh, Hh, B), "launch_us": dtc * 1e6,
                       "hbm_gbs": nbytes / dtc / 1e9, "hbm_frac": nbytes / dtc / 1e9 / hbm, "tflops": fl / dtc / 1e12,
                       "tensor_frac": fl / dtc / 1e12 / tflops})
    # the same kernels at the kernel-sweep size, where a launch moves enough data for bandwidth to matter
    for (Hh, Cc) in ((32, 16), (16, 32), (8, 64)):
        dtc, nbytes, fl, _ = conv_case(Hh, Cc, 4096)
        others.append({"kernel": "conv3x3_tc_kernel<%d> fwd %dx%d B=4096 (kernel-sweep size)" % (Cc, Hh, Hh),
                       "launch_us": dtc * 1e6, "hbm_gbs": nbytes / dtc / 1e9, "hbm_frac": nbytes / dtc / 1e9 / hbm,
                       "tflops": fl / dtc / 1e12, "tensor_frac": fl / dtc / 1e12 / tflops})
    torch.cuda.empty_cache()
    # batch-norm backward (sums + element-wise pass) on the largest map
    H, C = 32, 16
    per = 4 * B * H * H * C * 2
    n = max(8, int(400e6 // per) + 1)
    xs = [torch.randn(B, H * H, C, device="cuda").to(bf) for _ in range(n)]
    douts = [torch.randn_like(xs[0]) for _ in range(n)]
    dxs = [torch.empty_like(xs[0]) for _ in range(n)]
    g = torch.ones(C, device="cuda").to(bf)
    mean, invstd = torch.zeros(C, device="cuda"), torch.ones(C, device="cuda")
    dg, db = torch.empty(C, device="cuda"), torch.empty(C, device="cuda")
    scr = torch.zeros(binding.bn_scratch_elems(C), device="cuda")
    fns = [(lambda st, i=i: binding.bn_bwd(1, douts[i], xs[i], xs[i], g, mean, invstd, dxs[i], dg, db, scr, B, H * H, C, 1,
                                           st)) for i in range(n)]
    dtb = _time_back_to_back(torch, fns, s)
    nb = 7 * B * H * H * C * 2                               # sums read dout, out, x; the element-wise pass reads them again, writes dx
    others.append({"kernel": "bn_reduce_fast_kernel + bn_bwd_apply_fast_kernel (batch-norm backward) C=16 32x32 B=%d" % B,
                   "launch_us": dtb * 1e6, "hbm_gbs": nb / dtb / 1e9, "hbm_frac": nb / dtb / 1e9 / hbm})
    return roof, others


def max_over_ranks(values, dist, device):
    """Element-wise maximum over all ranks of a short list of durations (every rank gets the result); identity for a
    single process.  Replicas are independent, so the slowest one bounds the job."""
    import torch
    tt = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return [float(v) for v in tt]


def job_throughput(batch, steps, world, seconds):
    """Whole-job images/s of `world` independent replicas that each ran `steps` iterations of `batch` images."""
    return batch * steps * world / seconds


def main():
    args = parse()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    cfg = workload(args)
    K = len(cfg["split_after"]) + 1
    wl = "%s K=%d batch %d %s, synthetic CIFAR-shaped N(0,1) images, %d classes" % (
        args.net, K, cfg["batch"], cfg["precision"], cfg["num_classes"])

    if args.impl == "reference":
        if rank != 0:
            return 0
        # a step of this arm = one oracle iteration on the bounded sample (batch 8 of 128, ~0.55 s on 16 cores); the
        # requested steps are honoured up to 100, so that the run ends within a minute or two
        n = args.cpu_steps or min(max(args.steps, 1), 100)
        times = [time_oracle(cfg, args.cpu_batch, 1) for _ in range(min(args.warmup, 1))]   # one warm-up sample
        r = time_oracle(cfg, args.cpu_batch, n)
        out = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": "images/s", "n_gpus": 0,
               "steps": n, "warmup": len(times), "ms_per_step": 1e3 * r["seconds"] / n, "higher_is_better": True,
               "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
               "config": {"workload": wl, "sample": r["sample"]},
               "cpu_baseline": {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")},
               "e2e": {"value": r["value"], "unit": "images/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
        print(json.dumps(out))
        return 0

    import torch
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the DDG step has no CPU path")
    torch.cuda.set_device(local)
    from paper_1804_10574_b200 import binding, synth
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    streams = [torch.cuda.Stream() for _ in range(K)]
    o = cfg["opt"]
    net = binding.Ddg(cfg["layers"], cfg["split_after"], cfg["batch"], cfg["in_shape"], cfg["num_classes"],
                      precision=cfg["precision"], lr=o["lr"], momentum=o["momentum"], weight_decay=o["weight_decay"],
                      use_graph=not args.no_graph, streams=[s.cuda_stream for s in streams],
                      fuse_bn_apply=args.fuse_bn_apply, bn_fold=args.bn_fold)
    net.set_weights(synth.init_weights(cfg["layers"]))
    n_batches = K + 2
    host = [synth.batch(t, cfg["batch"], cfg["in_shape"], cfg["num_classes"]) for t in range(n_batches)]
    dev = [(torch.from_numpy(x).cuda(), torch.from_numpy(y).cuda()) for x, y in host]
    pinned = [(torch.from_numpy(x).pin_memory(), torch.from_numpy(y).pin_memory()) for x, y in host]
    warm = max(args.warmup, K - 1 + 3)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident throughput: inputs already in HBM, no host round trip inside the timed region ----
    for t in range(warm):
        net.step(*dev[t % n_batches], want_loss=False)
    net.sync()
    launches_per_step = net.last_step_launches()
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(streams[0])
    for t in range(args.steps):
        net.step(*dev[(warm + t) % n_batches], want_loss=False)
    net.sync()                       # all K streams drained; the end event then lands after every kernel of the region
    e1.record(streams[0])
    barrier()
    dt = e0.elapsed_time(e1) * 1e-3

    # ---- end to end through the public call with host buffers: H2D of x, y and D2H of the loss every step ----
    for t in range(3):
        net.step_host(*pinned[t % n_batches])
    barrier()
    n_e2e = max(10, args.steps // 4)
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(streams[0])
    for t in range(n_e2e):
        loss = net.step_host(*pinned[t % n_batches])
    net.sync()                       # the last iteration's backward sweeps and updates belong to the timed region
    f1.record(streams[0])
    barrier()
    dt_e2e = f0.elapsed_time(f1) * 1e-3
    # the same loop through the pipelined call: the host enqueues iteration t and reads the loss of iteration t-1, so it
    # never waits for the device inside an iteration; every iteration's inputs still come from pinned host memory and
    # every iteration's loss is still read by the host inside the timed region (the last one by ddg_pipelined_loss)
    for t in range(3):
        net.step_host_pipelined(*pinned[t % n_batches])
    net.pipelined_loss()
    barrier()
    h0, h1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    h0.record(streams[0])
    for t in range(n_e2e):
        net.step_host_pipelined(*pinned[t % n_batches])
    net.pipelined_loss()
    net.sync()
    h1.record(streams[0])
    barrier()
    dt_pipe = h0.elapsed_time(h1) * 1e-3
    # the sampler ran through both timed regions (device-resident and end-to-end): a 20-iteration region alone lasts
    # ~40 ms, too short for nvidia-smi's sampling period to land in it reliably
    clocks = sampler.stop()
    net.destroy()

    # ---- the same kernels with K = 1 (plain backpropagation, Section 3.2), same run, same batches ----
    k1 = None
    if K > 1 and not args.skip_k1:
        net1 = binding.Ddg(cfg["layers"], [], cfg["batch"], cfg["in_shape"], cfg["num_classes"],
                           precision=cfg["precision"], lr=o["lr"], momentum=o["momentum"], weight_decay=o["weight_decay"],
                           use_graph=not args.no_graph, streams=[streams[0].cuda_stream])
        net1.set_weights(synth.init_weights(cfg["layers"]))
        for t in range(max(args.warmup, 3)):
            net1.step(*dev[t % n_batches], want_loss=False)
        net1.sync()
        barrier()
        g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        n_k1 = max(10, args.steps // 2)
        g0.record(streams[0])
        for t in range(n_k1):
            net1.step(*dev[t % n_batches], want_loss=False)
        net1.sync()
        g1.record(streams[0])
        barrier()
        dt_k1 = max_over_ranks([g0.elapsed_time(g1) * 1e-3], dist, "cuda")[0]
        k1 = {"value": job_throughput(cfg["batch"], n_k1, world, dt_k1), "unit": "images/s", "ms_per_step": 1e3 * dt_k1 / n_k1,
              "steps": n_k1, "launches_per_step": int(net1.last_step_launches()),
              "what": "the same network, kernels and batches with K = 1 (plain backpropagation)"}
        net1.destroy()

    # ---- where the iteration's time sits: device time of each module's forward piece and backward + update piece
    # (the quantities of the method's cost model: forward sweeps in sequence, backward sweeps side by side), from a
    # short run of its own with the piece timer on, outside every timed region ----
    pieces = None
    if rank == 0 and not args.skip_k1:
        netp = binding.Ddg(cfg["layers"], cfg["split_after"], cfg["batch"], cfg["in_shape"], cfg["num_classes"],
                           precision=cfg["precision"], lr=o["lr"], momentum=o["momentum"], weight_decay=o["weight_decay"],
                           use_graph=not args.no_graph, streams=[s.cuda_stream for s in streams],
                           fuse_bn_apply=args.fuse_bn_apply, bn_fold=args.bn_fold, time_pieces=True)
        netp.set_weights(synth.init_weights(cfg["layers"]))
        fs, bs = [], []
        for t in range(warm + 9):
            netp.step(*dev[t % n_batches], want_loss=False)
            if t >= warm:
                f, b = netp.piece_times()
                fs.append(f)
                bs.append(b)
        netp.destroy()
        pieces = {"fwd_ms": [round(float(v), 4) for v in np.median(np.array(fs), axis=0)],
                  "bwd_upd_ms": [round(float(v), 4) for v in np.median(np.array(bs), axis=0)],
                  "what": "median device time per module of F_k and of B_k + U_k over 9 iterations run one at a time "
                          "(each drained before the next: no overlap between iterations, unlike the timed region)"}

    dt, dt_e2e, dt_pipe = max_over_ranks([dt, dt_e2e, dt_pipe], dist, "cuda")

    if rank == 0:
        peaks = {}
        try:
            peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
        except Exception:
            pass
        roof, roof_others = dominant_kernel_roofline(torch, binding, cfg, peaks, K)
        cpu = None
        if world == 1 and not args.skip_cpu:
            r = time_oracle(cfg, args.cpu_batch, args.cpu_steps or 20)   # ~10 s of host work
            cpu = {k: r[k] for k in ("value", "unit", "cores", "kind", "sample")}
        x_bytes = int(np.prod((cfg["batch"],) + tuple(cfg["in_shape"]))) * 4
        out = {"metric": METRIC, "value": job_throughput(cfg["batch"], args.steps, world, dt), "unit": "images/s", "n_gpus": world, "steps": args.steps,
               "warmup": warm, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16" if cfg["precision"] == "bf16" else "f32", "data": "synthetic",
               "config": {"workload": wl, "parallelism": "%d CUDA streams on one GPU%s" % (
                   K, "" if world == 1 else ", %d independent replicas" % world),
                   "cuda_graph": not args.no_graph,
                   "l2": "no flush: one iteration touches > 1 GB of activations, far above the 126 MB L2",
                   "final_loss": loss},
               "clocks": clocks, "gpu_launches": int(launches_per_step * args.steps),
               "launches_per_step": int(launches_per_step),
               "e2e": {"value": job_throughput(cfg["batch"], n_e2e, world, dt_e2e), "unit": "images/s",
                       "h2d_bytes_per_step": x_bytes + cfg["batch"] * 4, "d2h_bytes_per_step": 4, "steps": n_e2e},
               "e2e_pipelined": {"value": job_throughput(cfg["batch"], n_e2e, world, dt_pipe), "unit": "images/s",
                                 "h2d_bytes_per_step": x_bytes + cfg["batch"] * 4, "d2h_bytes_per_step": 4, "steps": n_e2e,
                                 "what": "ddg_step_host_pipelined: as e2e, but the host reads the loss of iteration t-1 "
                                         "while iteration t runs instead of waiting for iteration t's"},
               "k1_baseline": k1, "pieces": pieces, "roofline": roof, "roofline_others": roof_others, "cpu_baseline": cpu}
        if k1:
            out["k1_baseline"]["speedup_of_ddg"] = out["value"] / k1["value"]
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()
    return 0


if __name__ == "__main__":
    sys.exit(main())

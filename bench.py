"""Benchmark: SqueezeNet v1.0 forward, images/s.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
  python -m torch.distributed.run --nnodes=1 --nproc-per-node N ... bench.py --gpus N ...

A step is one forward of the whole network over one batch of synthetic images
(default: batch 256 per GPU, bf16 activations/kernels with fp32 accumulation on the
tensor cores).  Images are independent, so N GPUs run N replicas on their own batches
(weak scaling, no collective on the data path); the job's value is all images / the
slowest rank's device time.  Rank 0 prints one JSON line.
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

from paper_1611_07151_b200 import dist as D
from paper_1611_07151_b200 import synth

IMG = 227
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "dram_bytes_per_launch.txt")


def ncu_traffic_bytes(launch, dtype, batch):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch, from the committed table of single-pass ncu
    captures (lines: launch dtype batch bytes); None when the table has no line for this launch and configuration."""
    try:
        with open(TRAFFIC_TABLE) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 4 and not line.startswith("#") and parts[0] == launch and parts[1] == dtype \
                        and int(parts[2]) == batch:
                    return float(parts[3])
    except OSError:
        pass
    return None


METRIC = "squeezenet_v1.0_forward_images_per_s"
UNIT = "images/s"


# --------------------------------------------------------------------------- peaks
def measured_peaks():
    """Roofline denominators measured on this machine (written by the driver), else the fallback figures."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def fp32_ffma_peak_tflops(sm_count, sm_mhz):
    """FP32 pipe peak: SMs x 128 lanes x 2 flop x clock."""
    return sm_count * 128 * 2 * sm_mhz * 1e6 / 1e12


# ---------------------------------------------------------- algorithmic work per launch
def launch_work(batch, es):
    """name -> dict(flops, bytes) per forward, counting every tensor a launch must read or write once."""
    work = {}
    hw_out = {"conv1": 111}
    for name, cin, cout, k, s, pad, hw in synth.SQUEEZENET_CONVS:
        oh = (hw + 2 * pad - k) // s + 1
        flops = 2.0 * batch * oh * oh * cout * cin * k * k
        byts = es * batch * (hw * hw * cin + oh * oh * cout) + es * cout * cin * k * k + 4 * cout
        work[name] = {"flops": flops, "bytes": float(byts)}
    for name, c, h in (("pool1", 96, 111), ("pool4", 256, 55), ("pool8", 512, 27)):
        o = (h - 3) // 2 + 1
        work[name] = {"flops": 0.0, "bytes": float(es * batch * c * (h * h + o * o))}
    work["head"] = {"flops": 0.0, "bytes": float(batch * (es * 1000 * 169 + 8 * 1000))}
    # conv10, ReLU and the global average in one kernel: 512x13x13 in, 1000 means out; the softmax on its own
    work["conv10+avgpool"] = {"flops": work["conv10"]["flops"],
                              "bytes": float(batch * (es * 512 * 169 + 4 * 1000) + es * 1000 * 512 + 4 * 1000)}
    work["softmax"] = {"flops": 0.0, "bytes": float(batch * 8 * 1000)}
    # a whole fire layer in one kernel: input map in, both expands' output out, all kernels once
    for i in range(2, 10):
        f = "fire%d" % i
        cin, s_, hw = [(c, co, h) for nm, c, co, k, st, pd, h in synth.SQUEEZENET_CONVS if nm == f + "_sq"][0]
        e_ = [co for nm, c, co, *_ in synth.SQUEEZENET_CONVS if nm == f + "_e1"][0]
        work[f + "_fused"] = {"flops": work[f + "_sq"]["flops"] + work[f + "_e1"]["flops"] + work[f + "_e3"]["flops"],
                              "bytes": float(es * batch * hw * hw * (cin + 2 * e_) + es * (s_ * cin + 10 * e_ * s_) + 4 * (s_ + 2 * e_))}
    # repack of the stem's input (3 -> 4 layers, padded rows): an extra pass, counted at its real traffic
    work["conv1_pack"] = {"flops": 0.0, "bytes": float(batch * (IMG * IMG * 3 * 2 + 228 * 228 * 8))}
    # stem with its max-pool fused: the 96x111x111 map is never stored, only the pooled 96x55x55 one
    work["conv1+pool1"] = {"flops": work["conv1"]["flops"],
                           "bytes": float(es * batch * (IMG * IMG * 3 + 55 * 55 * 96) + es * 96 * 147 + 4 * 96)}
    # fire4's / fire8's expands with the following pool fused: squeeze map in, pooled half of the output out
    for fire, hw, ph, sq, e in ((4, 55, 27, 32, 128), (8, 27, 13, 64, 256)):
        for nm, k in (("fire%d_e1" % fire, 1), ("fire%d_e3" % fire, 3)):
            work[nm + "+pool"] = {"flops": work[nm]["flops"],
                                  "bytes": float(es * batch * (hw * hw * sq + ph * ph * e) + es * e * sq * k * k + 4 * e)}
    # both expands of a fire layer in one launch: squeeze map in once, both halves of the output
    for i in range(2, 10):
        f = "fire%d" % i
        for a, b, n in ((f + "_e1", f + "_e3", f + "_e1+e3"), (f + "_e1+pool", f + "_e3+pool", f + "_e1+e3+pool")):
            if a in work and b in work:
                sq = es * batch * [c for nm, c, *_ in synth.SQUEEZENET_CONVS if nm == f + "_e1"][0] * \
                    [hw for nm, *_, hw in synth.SQUEEZENET_CONVS if nm == f + "_e1"][0] ** 2
                work[n] = {"flops": work[a]["flops"] + work[b]["flops"], "bytes": work[a]["bytes"] + work[b]["bytes"] - sq}
    return work


# ------------------------------------------------------------------- clock sampling
class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs (read only)."""

    def __init__(self, index, period=0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {"hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
                 "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
                 "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
                 "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4)}
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_rank):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ------------------------------------------------------------------ oracle timings
def oracle_images_per_s(n_images, seed, repeats=1):
    """Times the CPU oracle, as it stands, on n_images of the workload.  Returns (images/s, threads)."""
    from oracle import ref
    x, params = synth.squeezenet_case(seed, n_images)
    t0 = time.perf_counter()
    for _ in range(repeats):
        ref.squeezenet(x, params)
    dt = time.perf_counter() - t0
    return n_images * repeats / dt, ref.max_threads()


def run_reference(args):
    """--impl reference: the oracle on the host cores, same metric/config, bounded sample per step."""
    rank, _local, world = D.env_world()
    if rank != 0:
        return
    from oracle import ref
    x1, params = synth.squeezenet_case(3, 1)
    t0 = time.perf_counter()
    ref.squeezenet(x1, params)
    t_img = time.perf_counter() - t0
    budget = 150.0 / max(1, args.steps + args.warmup)
    n_img = int(max(1, min(args.batch, budget // max(t_img, 1e-6))))
    x, _ = synth.squeezenet_case(3, n_img)
    for _ in range(args.warmup):
        ref.squeezenet(x, params)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        ref.squeezenet(x, params)
    dt = time.perf_counter() - t0
    value = n_img * args.steps / dt
    cores = ref.max_threads()
    sample = "%d of the %d images of the batch per step, full network, all host threads" % (n_img, args.batch)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": workload_name(args), "batch_per_gpu": args.batch, "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_batch1(B, ws, bs, x1, dtype, dev, prepacked=False, iters=300):
    """The paper's own regime: one image at a time.  Launch-latency bound; timed hot (back-to-back launches, and
    replays of a CUDA graph captured around the same call: every tensor stays in the L2) and cold (the L2 is
    overwritten before every forward, one forward per event pair, median and mean)."""
    import torch
    net1 = B.squeezenet_create(ws, bs, dtype, 1)
    if prepacked:
        B.squeezenet_set_stem_prepacked(net1, True)
    work = torch.empty(B.squeezenet_workspace_bytes(net1, 1), dtype=torch.uint8, device=dev)
    logits = torch.empty((1, 1000), dtype=torch.float32, device=dev)
    probs = torch.empty((1, 1000), dtype=torch.float32, device=dev)
    out = {"note": "batch 1; hot = inputs and activations resident in L2, cold = L2 overwritten before each forward"}
    for _ in range(5):
        B.squeezenet_forward(net1, x1, logits, probs, work, 1)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        B.squeezenet_forward(net1, x1, logits, probs, work, 1)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / iters
    out["eager"] = {"images_per_s": 1e3 / ms, "latency_us": ms * 1e3}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    cold = []
    for _ in range(40):
        flush.zero_()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        B.squeezenet_forward(net1, x1, logits, probs, work, 1)
        b.record()
        torch.cuda.synchronize()
        cold.append(a.elapsed_time(b) * 1e3)
    out["cold"] = {"latency_us_median": float(np.median(cold)), "latency_us_mean": float(np.mean(cold)), "forwards": len(cold)}
    del flush
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            B.squeezenet_forward(net1, x1, logits, probs, work, 1)
            with torch.cuda.graph(g, stream=side):
                B.squeezenet_forward(net1, x1, logits, probs, work, 1)
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        for _ in range(5):
            g.replay()
        torch.cuda.synchronize()
        e0.record()
        for _ in range(iters):
            g.replay()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / iters
        out["cuda_graph"] = {"images_per_s": 1e3 / ms, "latency_us": ms * 1e3}
    except Exception as exc:                      # graph capture is optional plumbing, not the product
        out["cuda_graph"] = {"error": str(exc)[:200]}
    assert B.sqn_check() == B.SQN_OK
    B.squeezenet_destroy(net1)
    return out


def layer_table(B, net, step, steps, batch, es, dtype_tag, peaks, sm_count, sm_mhz, stream):
    """Per-launch times of `steps` forwards (CUDA events recorded by the library on the launching stream) -> one
    record per launch with its algorithmic work, its bound and the achieved fraction of it.  bf16 fractions are
    against the burst tensor peak (`frac`; a launch lasts tens of microseconds) with the sustained figure beside
    it; HBM fractions against the measured copy bandwidth with the nominal 8 TB/s beside it."""
    import torch
    B.squeezenet_profile(net, steps)
    pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    pe0.record(stream)
    for i in range(steps):
        step(i)
    pe1.record(stream)
    torch.cuda.synchronize()
    ms_step = pe0.elapsed_time(pe1) / steps
    lnames, lms, nfwd = B.squeezenet_profile_read(net)
    B.squeezenet_profile(net, 0)
    bf16 = dtype_tag in ("bf16", "f16")          # (the 16-bit tensor-core paths: same MMA rate)
    pipe = peaks["bf16_tflops"] if bf16 else fp32_ffma_peak_tflops(sm_count, sm_mhz)
    pipe_sus = peaks["bf16_tflops_sustained"] if bf16 else pipe
    work = launch_work(batch, es)
    layers = []
    total_ms = sum(lms) / max(nfwd, 1)
    for n, ms_sum in zip(lnames, lms):
        ms = ms_sum / max(nfwd, 1)
        w = work.get(n, {"flops": 0.0, "bytes": 0.0})
        t_hbm = w["bytes"] / (peaks["hbm_gbs"] * 1e9)
        t_pipe = w["flops"] / (pipe * 1e12)
        bound = "hbm" if t_hbm >= t_pipe else ("tensor" if bf16 else "alu")
        rec = {"name": n, "ms": ms, "share": ms / total_ms if total_ms else 0.0, "bound": bound,
               "gbs": w["bytes"] / (ms * 1e-3) / 1e9 if ms > 0 else 0.0,
               "tflops": w["flops"] / (ms * 1e-3) / 1e12 if ms > 0 else 0.0,
               "frac": max(t_hbm, t_pipe) / (ms * 1e-3) if ms > 0 else 0.0,
               "bytes": w["bytes"], "flops": w["flops"]}
        if bound == "hbm":
            rec["frac_nominal_8tbs"] = rec["gbs"] / 8000.0
        elif bf16:
            rec["frac_sustained"] = rec["tflops"] / pipe_sus
        rec["meets_60pct"] = bool(rec["frac"] >= 0.6)
        layers.append(rec)
    return layers, ms_step, pipe, pipe_sus


def run_sweep(B, family="squeezenet"):
    """Every distinct conv shape of a workload (SqueezeNet v1.0, or the bottleneck-network family) at batch 1, 16, 64,
    256 in fp32 and bf16 (seed 4 recipe, values drawn on the device): median of ten single launches with the L2
    overwritten before each, and the mean of 20 back-to-back launches over rotating buffers."""
    import torch
    peaks = measured_peaks()
    dev = "cuda:0"
    torch.cuda.set_device(0)
    props = torch.cuda.get_device_properties(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    seen, rows = set(), []
    for name, cin, cout, k, s, pad, hw in (synth.SQUEEZENET_CONVS if family == "squeezenet" else synth.BOTTLENECK_CONVS):
        key = (cin, cout, k, s, pad, hw)
        if key in seen:
            continue
        seen.add(key)
        oh = (hw + 2 * pad - k) // s + 1
        for dtype, tag, es in ((B.SQN_F32, "f32", 4), (B.SQN_BF16, "bf16", 2)):
            tdt = torch.float32 if dtype == B.SQN_F32 else torch.bfloat16
            pipe_tf = peaks["bf16_tflops"] if dtype == B.SQN_BF16 else fp32_ffma_peak_tflops(
                props.multi_processor_count, 1965.0)
            for batch in (1, 16, 64, 256):
                x = torch.rand((batch, hw, hw, cin), device=dev, generator=gen).to(tdt)
                w = (torch.randn((cout, k, k, cin), device=dev, generator=gen) * (2.0 / (cin * k * k)) ** 0.5).to(tdt)
                b = torch.randn((cout,), device=dev, generator=gen) * 0.01
                out = torch.empty((batch, oh, oh, cout), device=dev, dtype=tdt)
                nb = B.conv_workspace_bytes(cin, cout, hw, hw, k, s, pad, batch, dtype)
                wsb = torch.empty(max(nb, 16), dtype=torch.uint8, device=dev)

                def call():
                    B.conv_forward_ex(x, w, b, out, cin, cout, hw, hw, k, s, pad, batch, dtype=dtype, workspace=wsb,
                                      workspace_bytes=nb)
                for _ in range(3):
                    call()
                times = []
                for _ in range(10):
                    flush.zero_()
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    call()
                    e1.record()
                    torch.cuda.synchronize()
                    times.append(e0.elapsed_time(e1))
                ms = float(np.median(times))
                # ... and back to back over a second buffer set (mean of 20 launches)
                x2, out2 = x.clone(), torch.empty_like(out)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(20):
                    if i & 1:
                        B.conv_forward_ex(x2, w, b, out2, cin, cout, hw, hw, k, s, pad, batch, dtype=dtype, workspace=wsb,
                                          workspace_bytes=nb)
                    else:
                        call()
                e1.record()
                torch.cuda.synchronize()
                ms_b2b = e0.elapsed_time(e1) / 20
                del x2, out2
                flops = 2.0 * batch * oh * oh * cout * cin * k * k
                byts = es * batch * (hw * hw * cin + oh * oh * cout) + es * cout * cin * k * k + 4 * cout
                t_hbm, t_pipe = byts / (peaks["hbm_gbs"] * 1e9), flops / (pipe_tf * 1e12)
                rows.append({"layer": name, "dtype": tag, "batch": batch, "ms": ms, "ms_back_to_back": ms_b2b, "tflops": flops / ms / 1e9,
                             "gbs": byts / ms / 1e6, "bound": "hbm" if t_hbm >= t_pipe else ("tensor" if tag == "bf16" else "alu"),
                             "frac": max(t_hbm, t_pipe) / (ms * 1e-3)})
                del x, w, out
    assert B.sqn_check() == B.SQN_OK
    print(json.dumps({"sweep": rows, "family": family, "peaks": peaks,
                      "note": "bf16 stem time includes its repack launches; ms: one launch, L2 flushed, median of 10; "
                              "ms_back_to_back: mean of 20 launches alternating two buffer sets"}))


def run_variants(B, batch):
    """The B200 analogue of the paper's thread-granularity study (Section III-D, Tables 1 and 3): every distinct conv
    shape (bf16, one batch) under every kernel variant that fits -- CTAs per SM (1 heavy or 2 light) x store chunk width
    (16/32/64 output layers) -- against the variant the library picks itself; optimal, pessimal and chosen per layer."""
    import torch
    dev = "cuda:0"
    torch.cuda.set_device(0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    seen, rows = set(), []
    for name, cin, cout, k, s, pad, hw in synth.SQUEEZENET_CONVS:
        key = (cin, cout, k, s, pad, hw)
        if key in seen or (k == 7):          # (the stem has one kernel variant)
            continue
        seen.add(key)
        oh = (hw + 2 * pad - k) // s + 1
        x = torch.rand((batch, hw, hw, cin), device=dev, generator=gen).to(torch.bfloat16)
        w = (torch.randn((cout, k, k, cin), device=dev, generator=gen) * (2.0 / (cin * k * k)) ** 0.5).to(torch.bfloat16)
        b = torch.randn((cout,), device=dev, generator=gen) * 0.01
        out = torch.empty((batch, oh, oh, cout), device=dev, dtype=torch.bfloat16)

        x2, out2 = x.clone(), torch.empty_like(out)

        def timed():
            """Mean of 20 back-to-back launches alternating two buffer sets (microseconds); None if the variant does not fit."""
            def call(i):
                if i & 1:
                    B.conv_forward_ex(x2, w, b, out2, cin, cout, hw, hw, k, s, pad, batch, dtype=B.SQN_BF16)
                else:
                    B.conv_forward_ex(x, w, b, out, cin, cout, hw, hw, k, s, pad, batch, dtype=B.SQN_BF16)
            try:
                for i in range(4):
                    call(i)
            except B.SqnError as e:
                assert e.status == B.SQN_ERR_UNSUPPORTED
                return None
            ts = []
            for _ in range(3):
                flush.zero_()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(20):
                    call(i)
                e1.record()
                torch.cuda.synchronize()
                ts.append(e0.elapsed_time(e1) / 20)
            return float(np.median(ts)) * 1e3

        os.environ.pop("SQN_TC_VARIANT", None)
        row = {"layer": name, "batch": batch, "chosen_us": timed(), "variants": {}}
        for ctas in (1, 2):
            for cw in (16, 32, 64):
                os.environ["SQN_TC_VARIANT"] = "%d,%d" % (ctas, cw)
                t = timed()
                if t is not None:
                    row["variants"]["%dx%d" % (ctas, cw)] = t
        os.environ.pop("SQN_TC_VARIANT", None)
        best = min(row["variants"].items(), key=lambda kv: kv[1])
        worst = max(row["variants"].items(), key=lambda kv: kv[1])
        row.update({"optimal": best[0], "optimal_us": best[1], "pessimal": worst[0], "pessimal_us": worst[1]})
        rows.append(row)
        del x, w, out, x2, out2
    assert B.sqn_check() == B.SQN_OK
    print(json.dumps({"variants": rows, "note": "variant = <CTAs per SM>x<store chunk width>; mean of 20 back-to-back launches "
                      "alternating two buffer sets, median of 3 such runs, microseconds; a missing variant does not fit the layer"}))


def run_kernel_case(B, name, batch, steps, dtype="bf16"):
    """One layer (or fire layer, or the fused head) of the network on its own (bf16 / f16 / f32), seed-4 recipe drawn on the device:
    `steps` back-to-back launches over rotating buffer sets larger than the L2 (mean), then single launches with the L2
    overwritten in between (median).  The small cases of the ncu captures under profiles/ are runs of this mode."""
    import torch
    dev = "cuda:0"
    torch.cuda.set_device(0)
    gen = torch.Generator(device=dev)
    gen.manual_seed(4)
    bf = {"bf16": torch.bfloat16, "f16": torch.float16, "f32": torch.float32}[dtype]
    code = {"bf16": B.SQN_BF16, "f16": B.SQN_F16, "f32": B.SQN_F32}[dtype]
    es = 4 if dtype == "f32" else 2
    convs = {n: (cin, cout, k, s, pad, hw) for n, cin, cout, k, s, pad, hw in synth.SQUEEZENET_CONVS}

    def conv_params(cin, cout, k):
        w = (torch.randn((cout, k, k, cin), device=dev, generator=gen) * (2.0 / (cin * k * k)) ** 0.5).to(bf)
        return w, torch.randn((cout,), device=dev, generator=gen) * 0.01

    sets = []
    if name.startswith("fire") and "_" not in name:
        cin, s_, _k, _s, _p, hw = convs[name + "_sq"]
        e = convs[name + "_e1"][1]
        wsq, bsq = conv_params(cin, s_, 1)
        w1, b1 = conv_params(s_, e, 1)
        w3, b3 = conv_params(s_, e, 3)
        per_set = batch * hw * hw * (cin + s_ + 2 * e) * es
        nsets = max(2, int(200e6 // per_set) + 1)
        for _ in range(nsets):
            sets.append((torch.rand((batch, hw, hw, cin), device=dev, generator=gen).to(bf),
                         torch.empty((batch, hw, hw, s_), device=dev, dtype=bf), torch.empty((batch, hw, hw, 2 * e), device=dev, dtype=bf)))

        def call(i):
            x, sc, out = sets[i % nsets]
            B.fire_forward(x, wsq, bsq, w1, b1, w3, b3, sc, out, cin, s_, e, e, hw, hw, batch, code)
        flops = 2.0 * batch * hw * hw * (cin * s_ + 10 * s_ * e)
        byts = float(es) * batch * hw * hw * (cin + 2 * e)
    else:
        base = name.split("+")[0]
        cin, cout, k, s_, pad, hw = convs[base]
        pool, avg = name.endswith("+pool") or name.endswith("+pool1"), name.endswith("+avgpool")
        oh = (hw + 2 * pad - k) // s_ + 1
        w, b = conv_params(cin, cout, k)
        nb = B.conv_workspace_bytes(cin, cout, hw, hw, k, s_, pad, batch, code)
        po = (oh - 3) // 2 + 1
        out_shape = (batch, cout) if avg else ((batch, po, po, cout) if pool else (batch, oh, oh, cout))
        per_set = batch * hw * hw * cin * es + int(np.prod(out_shape)) * es
        nsets = max(2, int(200e6 // per_set) + 1)
        for _ in range(nsets):
            sets.append((torch.rand((batch, hw, hw, cin), device=dev, generator=gen).to(bf),
                         torch.empty(out_shape, device=dev, dtype=torch.float32 if avg else bf),
                         torch.empty(max(nb, 16), dtype=torch.uint8, device=dev)))

        def call(i):
            x, out, wsb = sets[i % nsets]
            B.conv_forward_ex(x, w, b, out, cin, cout, hw, hw, k, s_, pad, batch, dtype=code, workspace=wsb,
                              workspace_bytes=nb, fuse_maxpool=pool, fuse_global_avgpool=avg)
        flops = 2.0 * batch * oh * oh * cout * cin * k * k
        byts = float(es) * batch * hw * hw * cin + (4.0 if avg else float(es)) * float(np.prod(out_shape))
    for i in range(5):
        call(i)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(steps):
        call(i)
    e1.record()
    torch.cuda.synchronize()
    mean_us = e0.elapsed_time(e1) / steps * 1e3
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    singles = []
    for i in range(min(steps, 20)):
        flush.zero_()
        a, c = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        call(i)
        c.record()
        torch.cuda.synchronize()
        singles.append(a.elapsed_time(c) * 1e3)
    assert B.sqn_check() == B.SQN_OK
    peaks = measured_peaks()
    print(json.dumps({"kernel_case": name, "dtype": dtype, "batch": batch, "steps": steps, "us_mean_back_to_back": mean_us,
                      "us_median_single_cold": float(np.median(singles)), "tflops": flops / mean_us / 1e6,
                      "gbs": byts / mean_us / 1e3, ("frac_ffma_peak" if dtype == "f32" else "frac_tensor_burst"): flops / mean_us / 1e6 / (fp32_ffma_peak_tflops(torch.cuda.get_device_properties(0).multi_processor_count, 1965) if dtype == "f32" else peaks["bf16_tflops"]),
                      "frac_hbm": byts / mean_us / 1e3 / peaks["hbm_gbs"], "buffer_sets": nsets}))


def workload_name(args):
    return "squeezenet_v1.0_forward_b%d_%s" % (args.batch, args.dtype)


# --------------------------------------------------------------------------- main
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=256, help="images per GPU per step")
    ap.add_argument("--dtype", default="bf16", choices=["bf16", "f16", "f32"])
    ap.add_argument("--e2e-steps", type=int, default=0, help="steps of the host-buffer loop (0: min(steps, 50))")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-batch1", action="store_true")
    ap.add_argument("--sweep", action="store_true", help="per-layer sweep of every conv shape instead of the network")
    ap.add_argument("--family", default="squeezenet", choices=["squeezenet", "bottleneck"],
                    help="--sweep: the workload whose conv shapes are swept (bottleneck: the 1x1 / 3x3 shapes of a residual network)")
    ap.add_argument("--variants", action="store_true", help="per-layer sweep of the bf16 kernel variants at --batch")
    ap.add_argument("--mma-rate", action="store_true", help="clocks per tcgen05.mma as a function of N (diagnostic)")
    ap.add_argument("--kernel", default=None, help="one layer on its own (bf16): a conv name (conv1, fire6_e3, ...), "
                    "NAME+pool, conv10+avgpool, or a fire layer (fire2 ... fire9)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    from paper_1611_07151_b200 import binding as B

    if args.sweep:
        run_sweep(B, args.family)
        return
    if args.variants:
        run_variants(B, args.batch)
        return
    if args.kernel:
        run_kernel_case(B, args.kernel, args.batch, args.steps, args.dtype)
        return
    if args.mma_rate:
        rows = []
        for rb in (32, 128):
            for n in (16, 32, 64, 96, 128, 192, 256):
                (issue, done), = B.sqn_selftest_mma_rate(n, rb, 1)
                rows.append({"row_bytes": rb, "N": n, "issuers": 1, "clocks_per_mma_issue": issue, "clocks_per_mma": done})
        for n in (16, 64, 128, 256):
            (i0, d0), (i1, d1) = B.sqn_selftest_mma_rate(n, 128, 2)
            rows.append({"row_bytes": 128, "N": n, "issuers": 2, "clocks_per_mma": [d0, d1]})
        assert B.sqn_check() == B.SQN_OK
        print(json.dumps({"mma_rate": rows, "note": "tcgen05.mma 128 x N x 16, bf16 operands in shared memory, issued back to "
                          "back by one elected thread per issuer warp on every SM; ideal N/2 clocks"}))
        return

    rank, local_rank, world = D.env_world()
    torch.cuda.set_device(local_rank)
    dev = "cuda:%d" % local_rank
    D.init("nccl")
    B.lib()                                     # raises if the CUDA library is missing: no other path exists

    dtype = {"bf16": B.SQN_BF16, "f16": B.SQN_F16, "f32": B.SQN_F32}[args.dtype]
    es = 4 if dtype == B.SQN_F32 else 2
    batch = args.batch
    bf16 = dtype == B.SQN_BF16          # (the stem's offline layouts and the fp32 sub-record go with the bf16 headline run)
    half = dtype != B.SQN_F32           # a 16-bit tensor-core path

    # ---- synthetic workload: U[0,1) images, He-normal kernels, N(0,.01) bias (seed 3 + rank)
    x, params = synth.squeezenet_case(3 + rank, batch)
    names = [n for n, *_ in synth.SQUEEZENET_CONVS]
    ws = [B.to_device(B.sqn_pack_weights_oihw_to_ohwi(params[n][0], dtype), dtype) for n in names]
    bs = [B.to_device(np.ascontiguousarray(params[n][1], dtype=np.float32)) for n in names]

    def pinned(a):
        t = torch.from_numpy(a)
        if half:
            t = t.view(torch.int16).view(torch.bfloat16 if bf16 else torch.float16)
        return t.pin_memory()

    x_pinned = pinned(B.sqn_pack_nchw_to_nhwc(x, dtype))              # [batch][227][227][3]: what a user's loader holds
    # Device-resident run: the bf16 stem reads operands reordered offline (input [batch][228][228][4], conv1's
    # kernels [96][7][8][4] with the bias folded in), so the forward launches no repack pass.
    if bf16:
        ws_dev = list(ws)
        ws_dev[0] = B.to_device(B.sqn_pack_stem_weights(*params["conv1"]), dtype)
        x_dev_host = pinned(B.sqn_pack_stem_input(x))
    else:
        ws_dev, x_dev_host = ws, x_pinned
    x32_one = np.ascontiguousarray(x[:1])
    del x
    inputs = [x_dev_host.to(dev), torch.flip(x_dev_host, dims=[0]).contiguous().to(dev)]   # rotated between steps

    net = B.squeezenet_create(ws_dev, bs, dtype, batch)
    if bf16:
        B.squeezenet_set_stem_prepacked(net, True)
    net_host = B.squeezenet_create(ws, bs, dtype, batch)            # host-buffer path: 3-layer images as they are
    work_bytes = B.squeezenet_host_workspace_bytes(net_host, batch)
    workspace = torch.empty(work_bytes, dtype=torch.uint8, device=dev)
    logits = torch.empty((batch, 1000), dtype=torch.float32, device=dev)
    probs = torch.empty((batch, 1000), dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()

    def step(i):
        B.squeezenet_forward(net, inputs[i & 1], logits, probs, workspace, batch)

    # ---- warm-up, then the timed region (device-resident inputs)
    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()
    assert B.sqn_check() == B.SQN_OK
    sampler = ClockSampler(physical_gpu_index(local_rank))
    D.barrier()
    torch.cuda.synchronize()
    launches0 = B.sqn_launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    ev0.record(stream)
    for i in range(args.steps):
        step(i)
    ev1.record(stream)
    torch.cuda.synchronize()
    D.barrier()
    gpu_launches = B.sqn_launch_count() - launches0
    ms_local = ev0.elapsed_time(ev1)
    status = B.sqn_check()
    assert status == B.SQN_OK, B.sqn_status_string(status)
    value, ms_total = D.job_throughput(batch * args.steps, ms_local, dev)

    # ---- the same steps once more with an event after every step: median beside the mean
    n_med = min(args.steps, 200)
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_med + 1)]
    evs[0].record(stream)
    for i in range(n_med):
        step(i)
        evs[i + 1].record(stream)
    torch.cuda.synchronize()
    per_step = [evs[i].elapsed_time(evs[i + 1]) for i in range(n_med)]

    # ---- per-launch times -> per-layer roofline.  One CUDA event per launch keeps a chained launch from starting
    # in the tail of the one before it (12 % on the whole forward at batch 256), so the events are recorded in a
    # further pass over the same steps and the timed region itself runs without.  The clock sampler runs across it.
    peaks = measured_peaks()
    props = torch.cuda.get_device_properties(local_rank)
    prof_steps = min(args.steps, 256)
    layers, ms_step_with_events, pipe_tf, pipe_sus = layer_table(
        B, net, step, prof_steps, batch, es, args.dtype, peaks, props.multi_processor_count, 1965.0, stream)
    clocks = sampler.stop()
    top = max(layers, key=lambda l: l["ms"])
    if top["bound"] == "hbm":
        roof = {"bound": "hbm", "achieved": top["gbs"], "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac_nominal_8tbs": top["gbs"] / 8000.0}
    else:
        roof = {"bound": top["bound"], "achieved": top["tflops"], "peak": pipe_tf, "unit": "TFLOP/s"}
        if half:
            roof["peak_kind"] = ("burst (a launch lasts %.0f us at full clocks); sustained peak %.1f beside it"
                                 % (top["ms"] * 1e3, pipe_sus))
            roof["frac_sustained"] = top["tflops"] / pipe_sus
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"] = ncu_traffic_bytes(top["name"], args.dtype, batch)
    if not half:
        kname = "conv_f32_kernel"
    elif "_fused" in top["name"] or ("_e1+e3" in top["name"] and "+pool" not in top["name"]):
        kname = "fire_fused_kernel"
    elif "+avgpool" in top["name"]:
        kname = "conv_head_kernel"
    else:
        kname = "conv_pool_kernel" if "+pool" in top["name"] else "conv_tc_kernel"
    roof["kernel"] = kname + "[%s]" % top["name"]
    roof["peak_source"] = "of " + peaks["source"]
    roof["launch_ms"] = top["ms"]
    roof["share_of_step"] = top["share"]
    roof["timing"] = ("CUDA events around every launch, %d steps run after the timed region; with the events "
                      "a step takes %.4f ms (launches no longer overlap the tail of the one before)"
                      % (prof_steps, ms_step_with_events))
    sum_bound_ms = sum(l["frac"] * l["ms"] for l in layers)
    roof["whole_step_frac_of_layer_bounds"] = sum_bound_ms / (ms_local / args.steps)     # against the timed step

    # ---- end to end: host buffers in, host buffers out, through the C ABI (copies inside the timed region)
    e2e_steps = args.e2e_steps or min(args.steps, 50)
    out_host = torch.empty((2, batch, 1000), dtype=torch.float32).pin_memory()
    for i in range(3):
        B.squeezenet_forward_host(net_host, x_pinned, out_host[0], out_host[1], workspace, batch)
    torch.cuda.synchronize()
    D.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for i in range(e2e_steps):
        B.squeezenet_forward_host(net_host, x_pinned, out_host[0], out_host[1], workspace, batch)
    e1.record(stream)
    torch.cuda.synchronize()
    D.barrier()
    e2e_value, _ = D.job_throughput(batch * e2e_steps, e0.elapsed_time(e1), dev)
    h2d = batch * IMG * IMG * 3 * es
    d2h = 2 * batch * 1000 * 4
    assert abs(float(out_host[1].sum()) - batch) < 1e-2 * batch     # probabilities came back
    # the host-buffer forward and the device-resident one classify the batch alike
    step(0)
    torch.cuda.synchronize()
    same_top1 = float((out_host[0].argmax(1) == logits.cpu().argmax(1)).float().mean())

    batch1 = None
    f32_record = None
    if rank == 0 and world == 1 and not args.no_batch1:
        batch1 = run_batch1(B, ws_dev, bs, inputs[0][:1].contiguous(), dtype, dev, prepacked=bf16)
        if bf16:
            # the exact path (fp32 storage and FFMA arithmetic): the same kernels packed as fp32
            ws32 = [B.to_device(B.sqn_pack_weights_oihw_to_ohwi(params[n][0], B.SQN_F32), B.SQN_F32) for n in names]
            x32 = B.to_device(B.sqn_pack_nchw_to_nhwc(x32_one, B.SQN_F32), B.SQN_F32)
            batch1["f32"] = run_batch1(B, ws32, bs, x32, B.SQN_F32, dev)
            # ... and at the bench's batch: images/s and the per-launch fractions of the FP32 pipe peak
            fb = min(batch, 256)
            net32 = B.squeezenet_create(ws32, bs, B.SQN_F32, fb)
            work32 = torch.empty(B.squeezenet_workspace_bytes(net32, fb), dtype=torch.uint8, device=dev)
            xin32 = inputs[0][:fb, :IMG, :IMG, :3].float().contiguous()

            def step32(i):
                B.squeezenet_forward(net32, xin32, logits[:fb], probs[:fb], work32, fb)
            for i in range(3):
                step32(i)
            torch.cuda.synchronize()
            n32 = 10
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(n32):
                step32(i)
            b.record(stream)
            torch.cuda.synchronize()
            ms32 = a.elapsed_time(b) / n32
            l32, _, pipe32, _ = layer_table(B, net32, step32, n32, fb, 4, "f32", peaks, props.multi_processor_count,
                                            clocks["sm_mhz"] or 1965.0, stream)
            f32_record = {"images_per_s": fb / (ms32 * 1e-3), "ms_per_step": ms32, "batch": fb, "steps": n32,
                          "ffma_peak_tflops": pipe32,
                          "layers": [{"name": l["name"], "ms": round(l["ms"], 6), "bound": l["bound"],
                                      "frac": round(l["frac"], 4), "meets_60pct": l["meets_60pct"]} for l in l32]}
            assert B.sqn_check() == B.SQN_OK
            B.squeezenet_destroy(net32)
            del ws32, work32, xin32

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import ref
        v1, cores = oracle_images_per_s(1, 3)
        n = int(min(64, max(2, 15.0 * v1)))
        v, cores = oracle_images_per_s(n, 3)
        ref.set_threads(1)
        v_single, _ = oracle_images_per_s(1, 3)
        ref.set_threads(cores)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": "%d of the %d images of one batch, full network, double accumulation" % (n, batch),
               "single_thread_images_per_s": v_single}

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_total / args.steps,
                "ms_per_step_median": float(np.median(per_step)), "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": args.dtype, "data": "synthetic",
                "config": {"workload": workload_name(args), "batch_per_gpu": batch, "global_batch": batch * world,
                           "image": "227x227x3", "parallelism": "replicas, batch sharded by image, no collective",
                           "input_layout": ("device-resident run: stem operands reordered offline ([228][228][4] images, "
                                            "[96][7][8][4] kernels); e2e: [227][227][3] images, repacked on the device")
                           if bf16 else "[227][227][3]",
                           "l2": "per-step activations (%.1f GB) exceed the 126 MB L2; two input batches alternate"
                                 % (B.squeezenet_workspace_bytes(net, batch) / 1e9)},
                "clocks": clocks,
                "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                        "steps": e2e_steps, "top1_same_as_device_resident": same_top1},
                "gpu_launches": int(gpu_launches),
                "roofline": roof,
                "cpu_baseline": cpu,
                "batch1": batch1,
                "f32": f32_record,
                "layers": [{k: (round(v, 6) if isinstance(v, float) else v) for k, v in l.items()} for l in layers]}
        print(json.dumps(line), flush=True)
    B.squeezenet_destroy(net)
    B.squeezenet_destroy(net_host)


if __name__ == "__main__":
    main()

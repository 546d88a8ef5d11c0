#!/usr/bin/env python
"""Benchmark of the hybrid attention layer on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

A step is one gformer_hybrid_attn call (all heads: windowed + linear, merged) on one batch of
synthetic Q, K, V.  Default workload: the long-sequence layer B=1, H=32, N=32768, d=128,
w=512, bf16 (6 windowed + 26 linear heads).  Every (batch, head) pair is an independent
unit, so with N GPUs each rank runs its own batch element (weak scaling, no collective on
the data path); rank 0 prints one JSON line.

--impl reference times the fp64 CPU oracle on the host cores, on a bounded sample of the
same workload (the first tokens of every head); it is a deliberately slow reference.

Other workloads (--workload): gpt2s, prefill4k, self32k (the bidirectional layer), decode256,
sweep5 (the 32 points of the fixed-65536-token sweep, one JSON line).  --kernel-only linear|window
runs only that head group's kernel a few times (a small driver for profilers).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "hybrid_attention_tokens_per_s"
UNIT = "tokens/s"
# oracle samples: the first tokens of every head of the workload
CPU_BASELINE_TOKENS = 32768  # cpu_baseline leg: a few seconds of fp64 work at d=128 (3 s on 16 cores)
REFERENCE_STEP_TOKENS = 4096  # --impl reference: about 1 s per step

WORKLOADS = {
    "long32k": dict(B=1, H=32, N=32768, d=128, w=512, seed=2),
    "gpt2s": dict(B=8, H=12, N=2048, d=64, w=128, seed=1),
    "prefill4k": dict(B=64, H=16, N=4096, d=64, w=256, seed=3),
    # the bidirectional ("self") layer on the long-sequence shape: two-sided windowed heads, global linear heads
    "self32k": dict(B=1, H=32, N=32768, d=128, w=512, seed=2, self_layer=True),
    # token-by-token decoding after a 4096-token prefill: a step = `steps` decode steps of the batch
    "decode256": dict(B=64, H=16, N=4096, d=64, w=256, seed=3, decode_steps=256),
    # the 32 points of the sweep at 65 536 tokens per launch (N, d, w vary; H = 16): one JSON line
    "sweep5": dict(sweep=True, H=16, seed=4),
}
NOMINAL_HBM_GBS = 8000.0  # the figure the target is phrased against; fractions of it are printed beside the measured ones


# ---- the multi-GPU contract ("replicas only"): every rank runs its own batch of the same shape on
# its own GPU, nothing is exchanged on the data path; the job's time is the slowest rank's and its
# throughput counts every rank's tokens.
def replica_seed(c, rank):
    """Seed of rank `rank`'s synthetic inputs (different data, same shapes)."""
    return c["seed"] + 1000 * rank


def max_over_ranks(values, dist, device):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    if dist is None:
        return [float(v) for v in values]
    import torch

    t = torch.tensor([float(v) for v in values], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_throughput(world, units_per_rank_per_step, steps, slowest_ms):
    """Whole-job units per second: all ranks' units over the slowest rank's time."""
    return world * units_per_rank_per_step * steps / (slowest_ms * 1e-3)


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def recorded_traffic(workload):
    """DRAM bytes per launch of the workload's kernels ({kernel: bytes}) from the committed ncu captures, if recorded."""
    p = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f).get(workload)
    return None


def l2_bytes(device_index):
    """Size of the L2 cache of the device (126 MB on a B200)."""
    import torch

    return int(torch.cuda.get_device_properties(device_index).L2_cache_size)


def rotation_sets(set_bytes, l2):
    """How many independent (Q, K, V, O) buffer sets a timed loop rotates through so that its traffic
    is real HBM traffic: one when a set alone exceeds the L2, else at least four and at least twice
    the L2 in total."""
    if set_bytes > l2:
        return 1
    return max(4, -(-2 * l2 // set_bytes))


def algorithmic_bytes(c):
    """Read Q, K, V once and write O once (bf16)."""
    return 4 * c["B"] * c["H"] * c["N"] * c["d"] * 2


class ClockSampler:
    """SM clock and throttle reasons sampled every 2 ms through NVML from a thread of this process,
    between start() and stop(): the samples lie inside the timed region, and the GPU is never idle
    waiting for a sampler to come up (an idle GPU changes its clocks).  Falls back to an
    `nvidia-smi -lms 100` child process when the NVML binding is missing."""

    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASON_BITS = {"sw_power_cap": 0x4, "hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20,
                   "hw_thermal_slowdown": 0x40}

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.samples = []
        self.thread = None
        self.stop_flag = False
        self.nvml = None
        self.handle = None
        self.file = None
        self.proc = None
        try:
            import pynvml

            pynvml.nvmlInit()
            # CUDA_VISIBLE_DEVICES may renumber the devices: go through the PCI bus id
            import torch

            bus = torch.cuda.get_device_properties(gpu_index).pci_bus_id if hasattr(
                torch.cuda.get_device_properties(gpu_index), "pci_bus_id") else None
            self.handle = pynvml.nvmlDeviceGetHandleByIndex(gpu_index)
            if bus is not None:
                for i in range(pynvml.nvmlDeviceGetCount()):
                    h = pynvml.nvmlDeviceGetHandleByIndex(i)
                    if pynvml.nvmlDeviceGetPciInfo(h).bus == bus:
                        self.handle = h
                        break
            self.nvml = pynvml
        except Exception:
            self.nvml = None

    def _loop(self):
        nv, h = self.nvml, self.handle
        while not self.stop_flag:
            try:
                self.samples.append((nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM),
                                     nv.nvmlDeviceGetCurrentClocksEventReasons(h)))
            except Exception:
                break
            time.sleep(0.002)

    def start(self):
        if self.nvml is not None:
            import threading

            self.thread = threading.Thread(target=self._loop, daemon=True)
            self.thread.start()
            return
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=self.file, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.nvml is not None:
            self.stop_flag = True
            if self.thread is not None:
                self.thread.join(timeout=2)
            if self.samples:
                sm = sorted(c for c, _ in self.samples)
                bits = 0
                for _, r in self.samples:
                    bits |= int(r)
                try:
                    smax = self.nvml.nvmlDeviceGetMaxClockInfo(self.handle, self.nvml.NVML_CLOCK_SM)
                except Exception:
                    smax = None
                out.update(sm_mhz=float(sm[len(sm) // 2]), sm_max_mhz=float(smax) if smax else None,
                           reasons=sorted(n for n, b in self.REASON_BITS.items() if bits & b),
                           samples=len(sm), source="NVML every 2 ms, warm-up and timed region")
            return out
        if self.proc is None:
            return out
        self.proc.terminate()  # the exact child started above
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.file.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1]))
                smax.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(names, parts[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            sm.sort()
            out.update(sm_mhz=sm[len(sm) // 2], sm_max_mhz=max(smax), reasons=sorted(reasons), samples=len(sm),
                       source="nvidia-smi -lms 100")
        return out


def oracle_sample_rate(c, sample_tokens):
    """Times the oracle on the first `sample_tokens` tokens of every head; tokens/s."""
    import torch

    import oracle
    from paper_2412_19829_b200 import synth

    n = min(c["N"], sample_tokens)
    q, k, v = synth.qkv(c["B"], c["H"], n, c["d"], "bf16", c["seed"])
    a = [t.to(torch.float64).numpy() for t in (q, k, v)]
    h0 = oracle.default_h_sparse(c["H"])
    t0 = time.perf_counter()
    (oracle.hybrid_attn_self if c.get("self_layer") else oracle.hybrid_attn)(a[0], a[1], a[2], c["w"], h_sparse=h0)
    dt = time.perf_counter() - t0
    return c["B"] * n / dt, dt, n, oracle.num_threads()


def oracle_decode_rate(c, steps):
    """Times `steps` oracle decode steps of the batch on a state whose ring is full; tokens/s."""
    import torch

    import oracle
    from paper_2412_19829_b200 import synth

    B, H, d, w = c["B"], c["H"], c["d"], c["w"]
    st = oracle.DecodeState(B, H, d, w, oracle.default_h_sparse(H))
    st.t = c["N"]  # the ring counts as full; zero contents cost the same arithmetic as any other
    tq, tk, tv = [t.to(torch.float64).numpy() for t in synth.decode_tokens(steps, B, H, d, "bf16", c["seed"])]
    t0 = time.perf_counter()
    for t in range(steps):
        oracle.decode_step(tq[t], tk[t], tv[t], st)
    dt = time.perf_counter() - t0
    return B * steps / dt, dt, steps, oracle.num_threads()


def run_reference(args, c, rank):
    if rank != 0:
        return
    import oracle  # noqa: F401  (CPU oracle: the reference arm of this benchmark)

    if "decode_steps" in c:
        n_steps = 16
        for _ in range(args.warmup):
            oracle_decode_rate(c, n_steps)
        times = [oracle_decode_rate(c, n_steps)[1] for _ in range(args.steps)]
        mean = sum(times) / len(times)
        value = c["B"] * n_steps / mean
        cores = oracle.num_threads()
        line = {
            "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, **{k: c[k] for k in ("B", "H", "d", "w")},
                       "h_sparse": oracle.default_h_sparse(c["H"]), "decode_steps_per_step": n_steps},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{n_steps} decode steps of the batch on a full ring per step, fp64"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0,
        }
        print(json.dumps(line), flush=True)
        return

    for _ in range(args.warmup):
        oracle_sample_rate(c, REFERENCE_STEP_TOKENS)
    times = []
    n = cores = 0
    for _ in range(args.steps):
        _, dt, n, cores = oracle_sample_rate(c, REFERENCE_STEP_TOKENS)
        times.append(dt)
    mean = sum(times) / len(times)
    value = c["B"] * n / mean
    sample = f"first {n} tokens of each of the {c['B'] * c['H']} heads per step, fp64, OpenMP over heads"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.workload, **{k: c[k] for k in ("B", "H", "N", "d", "w")},
                   "h_sparse": oracle.default_h_sparse(c["H"]), "sampled_tokens": n},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, c, rank, world, local_rank):
    import torch

    from paper_2412_19829_b200 import binding as gf
    from paper_2412_19829_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    h0 = gf.default_h_sparse(c["H"])
    B, H, N, d, w = c["B"], c["H"], c["N"], c["d"], c["w"]

    q, k, v = synth.qkv(B, H, N, d, "bf16", replica_seed(c, rank))
    hq, hk, hv = [t.pin_memory() for t in (q, k, v)]
    ho = torch.empty_like(hq).pin_memory()
    dq, dk, dv = [t.cuda() for t in (hq, hk, hv)]
    do = torch.empty_like(dq)
    favor = args.phi == "favor"
    Wd = synth.favor_projection(H - h0, d, seed=c["seed"], orthogonal=True, dtype="bf16").cuda() if favor else None
    ws = gf.Workspace.for_problem(B, H, N, d, w, h0, phi=gf.GF_PHI_FAVOR_POS if favor else gf.GF_PHI_ELU1)
    stream = torch.cuda.Stream()

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    self_layer = bool(c.get("self_layer"))
    base_layer = gf.hybrid_attn_self if self_layer else gf.hybrid_attn

    def layer(*a, **kw):
        return base_layer(*a, W=Wd, **kw)

    # Inputs that fit the L2 are rotated over several buffer sets, so that every step reads its
    # inputs from HBM; the L2-resident figure (one set, back to back) is reported beside it.
    l2 = l2_bytes(local_rank)
    set_bytes = 4 * B * H * N * d * 2
    n_sets = rotation_sets(set_bytes, l2)
    sets = [(dq, dk, dv, do)] + [tuple(t.clone() for t in (dq, dk, dv, do)) for _ in range(n_sets - 1)]
    turn = [0]

    def step():
        q_, k_, v_, o_ = sets[turn[0] % n_sets]
        turn[0] += 1
        layer(q_, k_, v_, w, h_sparse=h0, out=o_, ws=ws, stream=stream)

    def step_resident():
        layer(dq, dk, dv, w, h_sparse=h0, out=do, ws=ws, stream=stream)

    if args.kernel_only:  # a small driver for profilers: that head group's kernel alone, a few launches
        if args.kernel_only == "linear":
            lq, lk, lv, lo_ = [t[:, h0:].contiguous() for t in (dq, dk, dv, do)]
            ws_l = gf.Workspace.for_problem(B, H - h0, N, d, 1, 0)
            run = (lambda: gf.hybrid_attn_self(lq, lk, lv, w, h_sparse=0, out=lo_, ws=ws_l, stream=stream)) if self_layer \
                else (lambda: gf.causal_linear_attn(lq, lk, lv, out=lo_, ws=ws_l, stream=stream))
        else:
            wq, wk, wv, wo_ = [t[:, :h0].contiguous() for t in (dq, dk, dv, do)]
            run = (lambda: gf.window_attn_self(wq, wk, wv, w, out=wo_, ws=ws, stream=stream)) if self_layer \
                else (lambda: gf.window_attn(wq, wk, wv, w, out=wo_, ws=ws, stream=stream))
        for _ in range(max(args.warmup, 1) + args.steps):
            run()
        stream.synchronize()
        print(json.dumps({"kernel_only": args.kernel_only, "workload": args.workload, "launches": max(args.warmup, 1) + args.steps}))
        return

    # End to end, the way a caller would stream batches through the layer: two sets of device
    # buffers, the host-to-device copy of step i+1 and the device-to-host copy of step i-1 run on
    # streams of their own beside the layer call of step i (the link is full duplex and the copy
    # engines are separate from the SMs).  Every step still copies its own Q, K, V in from pinned
    # memory and its own output back; the timed region runs from the first copy to the last one.
    def timed_e2e_pipelined(steps):
        sets = [(dq, dk, dv, do), tuple(torch.empty_like(t) for t in (dq, dk, dv, do))]
        hos = [ho, torch.empty_like(ho).pin_memory()]
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        ev_in = [torch.cuda.Event() for _ in range(steps)]
        ev_done = [torch.cuda.Event() for _ in range(steps)]
        ev_out = [torch.cuda.Event() for _ in range(steps)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t0.record(s_in)
        for i in range(steps):
            q_, k_, v_, o_ = sets[i % 2]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_done[i - 2])  # the layer call that last read this input set
                q_.copy_(hq, non_blocking=True)
                k_.copy_(hk, non_blocking=True)
                v_.copy_(hv, non_blocking=True)
                ev_in[i].record(s_in)
            stream.wait_event(ev_in[i])
            if i >= 2:
                stream.wait_event(ev_out[i - 2])  # the copy that last read this output buffer
            layer(q_, k_, v_, w, h_sparse=h0, out=o_, ws=ws, stream=stream)
            ev_done[i].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_done[i])
                hos[i % 2].copy_(o_, non_blocking=True)
                ev_out[i].record(s_out)
        t1.record(s_out)
        s_out.synchronize()
        stream.synchronize()
        barrier()
        return t0.elapsed_time(t1)

    def step_e2e():
        with torch.cuda.stream(stream):
            dq.copy_(hq, non_blocking=True)
            dk.copy_(hk, non_blocking=True)
            dv.copy_(hv, non_blocking=True)
        step()
        with torch.cuda.stream(stream):
            ho.copy_(do, non_blocking=True)

    def timed(fn, steps):
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        barrier()
        evs[0].record(stream)
        for i in range(steps):
            fn()
            evs[i + 1].record(stream)
        stream.synchronize()
        barrier()
        total_ms = evs[0].elapsed_time(evs[-1])
        per = [evs[i].elapsed_time(evs[i + 1]) for i in range(steps)]
        return total_ms, per

    # clocks are sampled from the first warm-up step to the end of the timed region: the GPU is
    # under the benchmark's own load for all of it
    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    if sampler:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        step()
    stream.synchronize()
    if ws.last_device_status(stream) != gf.GF_OK:
        raise SystemExit("device-side wait timed out during warm-up")
    n0 = gf.launch_count()
    total_ms, per = timed(step, args.steps)
    launches = gf.launch_count() - n0
    if sampler:
        clocks = sampler.stop()
    if ws.last_device_status(stream) != gf.GF_OK:
        raise SystemExit("device-side wait timed out during the timed region")

    # Sustained figure: at least a second of back-to-back steps with the clocks sampled throughout
    # (a 1 kW part settles below its boost clock under a long load; time x clock tells the two apart).
    sustained = None
    if not args.no_sustained:  # every rank runs it (the timing helper holds a barrier); rank 0 samples the clocks
        n_long = max(args.steps, int(1.2e3 / max(total_ms / args.steps, 1e-3)))
        s2 = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
        if s2:
            s2.start()
        long_ms, _ = timed(step, n_long)
        (long_ms,) = max_over_ranks([long_ms], dist, "cuda")
        if s2:
            ck = s2.stop()
            sustained = {"steps": n_long, "seconds": long_ms * 1e-3, "ms_per_step": long_ms / n_long,
                         "sm_mhz_median": ck.get("sm_mhz"), "reasons": ck.get("reasons"),
                         "clock_samples": ck.get("samples"),
                         "ms_x_mhz": (long_ms / n_long) * ck["sm_mhz"] if ck.get("sm_mhz") else None}
    resident = None
    if n_sets > 1:
        for _ in range(3):
            step_resident()
        r_ms, _ = timed(step_resident, args.steps)
        resident = {"ms_per_step": r_ms / args.steps, "note": "one buffer set back to back: inputs stay in L2"}

    for _ in range(2):
        step_e2e()
    stream.synchronize()
    e2e_ms = timed_e2e_pipelined(args.steps)

    # The two kernels of a step, each timed alone over the same number of launches (B = 1 makes the
    # head slices contiguous): the dominant one carries the roofline entry.
    kern = {}
    if B == 1 and 0 < h0 < H and not favor:
        lq, lk, lv, lo_ = dq[:, h0:], dk[:, h0:], dv[:, h0:], do[:, h0:]
        wq, wk, wv, wo_ = dq[:, :h0], dk[:, :h0], dv[:, :h0], do[:, :h0]
        ws_l = gf.Workspace.for_problem(B, H - h0, N, d, 1, 0)
        if self_layer:
            lin = lambda: gf.hybrid_attn_self(lq, lk, lv, w, h_sparse=0, out=lo_, ws=ws_l, stream=stream)
            win = lambda: gf.window_attn_self(wq, wk, wv, w, out=wo_, ws=ws, stream=stream)
            names = ("linear_self kernels (reduce, sum, readout)", "window_tc_kernel (two-sided)")
        else:
            lin = lambda: gf.causal_linear_attn(lq, lk, lv, out=lo_, ws=ws_l, stream=stream)
            win = lambda: gf.window_attn(wq, wk, wv, w, out=wo_, ws=ws, stream=stream)
            names = ("linear_tc_kernel", "window_tc_kernel")
        for name, fn, heads in ((names[0], lin, H - h0), (names[1], win, h0)):
            for _ in range(3):
                fn()
            ms, _ = timed(fn, args.steps)
            kern[name] = {"ms_per_launch": ms / args.steps, "heads": heads,
                          "algorithmic_bytes": 4 * B * heads * N * d * 2}

    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], dist, "cuda")

    if rank == 0:
        value = job_throughput(world, B * N, args.steps, total_ms)
        e2e_value = job_throughput(world, B * N, args.steps, e2e_ms)
        peak, which = measured_peaks()
        abytes = algorithmic_bytes(c)
        mean_launch_s = (sum(per) / len(per)) * 1e-3
        step_gbs = abytes / mean_launch_s / 1e9
        tensor_bytes = B * H * N * d * 2
        if kern:
            dom = max(kern, key=lambda n: kern[n]["ms_per_launch"])
            dom_bytes = kern[dom]["algorithmic_bytes"]
            achieved = dom_bytes / (kern[dom]["ms_per_launch"] * 1e-3) / 1e9
            dom_desc = f"{dom} ({kern[dom]['heads']} of {H} heads), timed alone with CUDA events"
        else:
            dom, dom_bytes, achieved = "gformer_hybrid_attn step", abytes, step_gbs
            dom_desc = "whole step (both kernels)"
        traffic = recorded_traffic(args.workload) or {}
        step_traffic = sum(traffic.values()) if traffic and not favor and all(v is not None for v in traffic.values()) else None
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "B": B, "H": H, "N": N, "d": d, "w": w, "h_sparse": h0,
                       "phi": "positive random features (features of Q and K written to the workspace first)" if favor
                       else "elu + 1",
                       "global_batch": world * B, "seq_len": N,
                       "parallelism": "replicas only (one batch element per GPU, no collective)",
                       "l2": ("inputs larger than L2 (Q+K+V+O = %.0f MB per step, L2 %.0f MB)" % (set_bytes / 1e6, l2 / 1e6))
                       if n_sets == 1 else
                       ("inputs fit the L2 (%.0f MB of %.0f MB): steps rotate over %d buffer sets so that they read HBM; "
                        "the L2-resident figure is in l2_resident" % (set_bytes / 1e6, l2 / 1e6, n_sets))},
            # The headline figure is the whole layer's (what the target is phrased for): its algorithmic
            # bytes over the step time.  The kernel that takes most of the step, timed alone, is the
            # sub-entry `dominant_kernel`; `traffic` is the DRAM bytes of a step's kernels from the
            # committed ncu captures.
            "roofline": {"bound": "hbm", "achieved": step_gbs, "peak": peak, "unit": "GB/s",
                         "frac": step_gbs / peak, "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS,
                         "traffic": step_traffic, "peak_source": which + " copy bandwidth",
                         "algorithmic_bytes": abytes,
                         "kernel": "whole layer: every kernel of a step (see kernels), CUDA events around the step",
                         "tflops_algorithmic": algorithmic_flops(c, h0) / mean_launch_s / 1e12,
                         "dominant_kernel": {"name": dom, "how": dom_desc, "achieved": achieved, "frac": achieved / peak,
                                             "frac_of_nominal_8TBs": achieved / NOMINAL_HBM_GBS,
                                             "algorithmic_bytes": dom_bytes, "traffic": traffic.get(dom)},
                         "kernels": kern,
                         "step": {"achieved": step_gbs, "frac": step_gbs / peak,
                                  "frac_of_nominal_8TBs": step_gbs / NOMINAL_HBM_GBS, "algorithmic_bytes": abytes,
                                  "tflops_algorithmic": algorithmic_flops(c, h0) / mean_launch_s / 1e12}},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": 3 * tensor_bytes,
                    "d2h_bytes_per_step": tensor_bytes,
                    "how": "two buffer sets: the copies of neighbouring steps run on their own streams beside "
                           "the layer call; timed from the first copy in to the last copy out"},
            "gpu_launches": launches,
            "clocks": clocks,
            "step_ms_min": min(per), "step_ms_max": max(per),
        }
        if sustained:
            sustained["frac"] = abytes / (sustained["ms_per_step"] * 1e-3) / 1e9 / peak
            line["sustained"] = sustained
        if resident:
            resident["frac"] = abytes / (resident["ms_per_step"] * 1e-3) / 1e9 / peak
            line["l2_resident"] = resident
        if world == 1 and not args.no_cpu_baseline:
            rate, dt, n, cores = oracle_sample_rate(c, CPU_BASELINE_TOKENS)
            line["cpu_baseline"] = {
                "value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"first {n} tokens of each of the {B * H} heads, {dt:.1f} s of fp64 CPU work"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_decode(args, c, rank, world, local_rank):
    """Decode workload: prefill once (untimed), then time runs of `decode_steps` gformer_decode_step
    calls, once replayed from a CUDA graph captured over all of them and once launched one by one."""
    import torch

    from paper_2412_19829_b200 import binding as gf
    from paper_2412_19829_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    B, H, N, d, w, T = c["B"], c["H"], c["N"], c["d"], c["w"], c["decode_steps"]
    h0 = gf.default_h_sparse(H)
    q, k, v = synth.qkv(B, H, N, d, "bf16", replica_seed(c, rank))
    tq, tk, tv = synth.decode_tokens(T, B, H, d, "bf16", replica_seed(c, rank))
    htok = [t.pin_memory() for t in (tq, tk, tv)]
    dtok = [t.cuda() for t in htok]
    dout = torch.empty_like(dtok[0])
    hout = torch.empty_like(htok[0]).pin_memory()
    st = gf.DecodeState(B, H, d, w, h0)
    ws = gf.Workspace.for_problem(B, H, N, d, w, h0)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        gf.hybrid_attn(q.cuda(), k.cuda(), v.cuda(), w, h_sparse=h0, state_out=st, ws=ws, stream=stream)
    stream.synchronize()
    if ws.last_device_status(stream) != gf.GF_OK:
        raise SystemExit("device-side wait timed out during the prefill")

    def run_eager():
        st.t = N  # every run decodes the same positions N .. N + T - 1
        for t in range(T):
            gf.decode_step(dtok[0][t], dtok[1][t], dtok[2][t], st, out=dout[t], stream=stream)

    run_eager()
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        run_eager()

    def run_graph():
        with torch.cuda.stream(stream):
            graph.replay()

    def run_e2e():
        with torch.cuda.stream(stream):
            for dst, src in zip(dtok, htok):
                dst.copy_(src, non_blocking=True)
            graph.replay()
            hout.copy_(dout, non_blocking=True)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        e0.record(stream)
        for _ in range(steps):
            fn()
        e1.record(stream)
        stream.synchronize()
        barrier()
        return e0.elapsed_time(e1)

    sampler = ClockSampler(torch.cuda.current_device()) if rank == 0 else None
    if sampler:
        sampler.start()
    for _ in range(max(args.warmup, 3)):
        run_graph()
    n0 = gf.launch_count()
    total_ms = timed(run_graph, args.steps)
    clocks = sampler.stop() if sampler else None
    launches = gf.launch_count() - n0  # the graph replays the captured launches: count them below
    eager_ms = timed(run_eager, args.steps)

    # the same steps with per-sequence positions kept on the device (they advance from replay to
    # replay, the ring wraps): what a continuously batched server would replay
    t_seq = torch.full((B,), N, dtype=torch.int64, device="cuda")

    def run_ragged():
        for t in range(T):
            gf.decode_step_ragged(dtok[0][t], dtok[1][t], dtok[2][t], st, t_seq, out=dout[t], stream=stream)

    run_ragged()
    stream.synchronize()
    rgraph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(rgraph, stream=stream):
        run_ragged()

    def run_rgraph():
        with torch.cuda.stream(stream):
            rgraph.replay()

    run_rgraph()
    ragged_ms = timed(run_rgraph, args.steps)
    run_e2e()
    e2e_ms = timed(run_e2e, args.steps)
    total_ms, e2e_ms, eager_ms, ragged_ms = max_over_ranks([total_ms, e2e_ms, eager_ms, ragged_ms], dist, "cuda")
    if rank == 0:
        tokens = world * B * T * args.steps
        peak, which = measured_peaks()
        # per decode step: the ring's valid slots read once (K and V), S read and written, z and the
        # token's q, k, v, o
        ring = 2 * B * h0 * min(N, w) * d * 2
        state = 2 * B * (H - h0) * d * d * 4 + 2 * B * (H - h0) * d * 4
        step_bytes = ring + state + 4 * B * H * d * 2
        us_step = total_ms * 1e3 / (args.steps * T)
        achieved = step_bytes / (us_step * 1e-6) / 1e9
        line = {
            "metric": METRIC, "value": tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": args.workload, "B": B, "H": H, "d": d, "w": w, "h_sparse": h0, "prefill": N,
                       "decode_steps_per_step": T, "global_batch": world * B,
                       "parallelism": "replicas only (one batch per GPU, no collective)",
                       "l2": "state and ring (26 MB) stay in L2 between decode steps: an L2-resident number",
                       "launch": "one CUDA graph replay per step (all decode steps captured once)"},
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": None, "peak_source": which + " copy bandwidth",
                         "algorithmic_bytes": step_bytes, "kernel": "decode_step_kernel, one launch per decode step",
                         "us_per_decode_step_graph": us_step,
                         "us_per_decode_step_eager": eager_ms * 1e3 / (args.steps * T),
                         "us_per_decode_step_ragged_graph": ragged_ms * 1e3 / (args.steps * T)},
            "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": 3 * T * B * H * d * 2, "d2h_bytes_per_step": T * B * H * d * 2},
            "gpu_launches": args.steps * T if launches == 0 else launches,
            "clocks": clocks,
        }
        if world == 1 and not args.no_cpu_baseline:
            rate, dt, n, cores = oracle_decode_rate(c, 64)
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
                                    "sample": f"{n} decode steps of the batch on a full ring, {dt:.1f} s of fp64 CPU work"}
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


def run_sweep(args, c, rank, world, local_rank):
    """The 32 points of the sweep (65 536 tokens per launch, H = 16, default head split): per point the
    median launch time of `steps` launches and the fraction of the HBM roofline for the layer's
    algorithmic bytes; one JSON line.  Points whose tensors fit the L2 rotate over several buffer sets."""
    import statistics

    import torch

    from paper_2412_19829_b200 import binding as gf
    from paper_2412_19829_b200 import synth

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    if rank != 0:  # every point is one GPU's work: the other ranks of a multi-rank launch have nothing to do
        return
    stream = torch.cuda.Stream()
    peak, which = measured_peaks()
    l2 = l2_bytes(local_rank)
    sampler = ClockSampler(torch.cuda.current_device())
    sampler.start()
    points, total_ms, total_tokens, launches0 = [], 0.0, 0, gf.launch_count()
    for pt in synth.sweep_points():
        B, H, N, d, w = pt["B"], pt["H"], pt["N"], pt["d"], pt["w"]
        h0 = gf.default_h_sparse(H)
        g = torch.Generator(device="cuda").manual_seed(replica_seed(pt, rank))
        set_bytes = 4 * B * H * N * d * 2
        n_sets = rotation_sets(set_bytes, l2)
        sets = []
        for _ in range(n_sets):
            q, k, v = [torch.randn(B, H, N, d, device="cuda", generator=g).mul_(d ** -0.5).to(torch.bfloat16)
                       for _ in range(3)]
            sets.append((q, k, v, torch.empty_like(q)))
        ws = gf.Workspace.for_problem(B, H, N, d, w, h0)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        for i in range(max(args.warmup, 3)):
            q, k, v, o = sets[i % n_sets]
            gf.hybrid_attn(q, k, v, w, h_sparse=h0, out=o, ws=ws, stream=stream)
        stream.synchronize()
        evs[0].record(stream)
        for i in range(args.steps):
            q, k, v, o = sets[i % n_sets]
            gf.hybrid_attn(q, k, v, w, h_sparse=h0, out=o, ws=ws, stream=stream)
            evs[i + 1].record(stream)
        stream.synchronize()
        if ws.last_device_status(stream) != gf.GF_OK:
            raise SystemExit("device-side wait timed out")
        ms = statistics.median(evs[i].elapsed_time(evs[i + 1]) for i in range(args.steps))
        points.append({"N": N, "B": B, "d": d, "w": w, "h_sparse": h0, "ms": ms, "buffer_sets": n_sets,
                       "frac": set_bytes / (ms * 1e-3) / 1e9 / peak})
        total_ms += ms
        total_tokens += B * N
        del sets
    clocks = sampler.stop()
    fracs = sorted(p_["frac"] for p_ in points)
    line = {
        "metric": METRIC, "value": total_tokens / (total_ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic (seeded, generated on the device: timing only)",
        "config": {"workload": "sweep5", "points": len(points), "tokens_per_launch": 65536, "H": 16,
                   "step": "one launch of each of the 32 points (median launch times summed)",
                   "l2": "points that fit the L2 (%.0f MB) rotate over several buffer sets" % (l2 / 1e6)},
        "roofline": {"bound": "hbm", "peak": peak, "unit": "GB/s", "peak_source": which + " copy bandwidth",
                     "frac": fracs[len(fracs) // 2], "frac_worst": fracs[0], "frac_best": fracs[-1],
                     "achieved": fracs[len(fracs) // 2] * peak, "traffic": None,
                     "kernel": "whole layer per point (both kernels); frac is the median over the points"},
        "points": points, "gpu_launches": gf.launch_count() - launches0, "clocks": clocks,
    }
    print(json.dumps(line), flush=True)


def algorithmic_flops(c, h0):
    """Flops of the method itself: 4 d per (query, key) pair in the window, 4 d^2 per linear token."""
    B, H, N, d, w = c["B"], c["H"], c["N"], c["d"], c["w"]
    we = min(w, N)
    pairs = N * we - we * (we - 1) // 2
    if c.get("self_layer"):  # |i - j| < w: the causal band and its mirror share the diagonal
        pairs = 2 * pairs - N
    return B * (h0 * 4 * d * pairs + (H - h0) * 4 * N * d * d)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="long32k", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true", help="skip the one-second sustained run")
    ap.add_argument("--phi", choices=["elu1", "favor"], default="elu1",
                    help="feature map of the linear heads: elu + 1, or positive random features (seeded projections)")
    ap.add_argument("--kernel-only", choices=["linear", "window"], default=None,
                    help="run only that head group's kernel (no timing): a driver for profilers")
    args = ap.parse_args()
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    c = WORKLOADS[args.workload]
    if c.get("sweep"):
        if args.impl == "reference":
            if rank == 0:
                print(json.dumps({"impl": "reference", "unavailable": "the sweep workload has no reference arm: "
                                  "time the oracle on a single shape with --workload long32k/gpt2s/prefill4k"}))
            return
        run_sweep(args, c, rank, world, local_rank)
    elif args.impl == "reference":
        run_reference(args, c, rank)
    elif "decode_steps" in c:
        run_decode(args, c, rank, world, local_rank)
    else:
        run_ours(args, c, rank, world, local_rank)


if __name__ == "__main__":
    main()

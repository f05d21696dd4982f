#!/usr/bin/env python
"""Benchmark of the attention hot path: one step = forward + backward (delta, dQ, dK, dV)
over one batch of the GPT-2-small-shaped causal workload (B=16, H=12, N=1024, d=64, BF16).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--mode 0|1] [--impl ours|reference]
                  [--scaling weak|strong] [--context-libs]

Prints one JSON line (rank 0).  Metric: attention fwd+bwd TFLOP/s with the FLOP convention
fwd 4*Pi*d, bwd 10*Pi*d, Pi = B*H*N^2/2 score pairs for causal attention.
Multi-GPU: the (batch, head) problems are independent, so there is no data-path collective.
--scaling weak (default): every rank runs the whole batch shape on its own GPU; --scaling strong: one
batch is split over the ranks by contiguous (batch, head) ranges.  Time = max over ranks.
--context-libs adds, under its own key, the same workload timed through the attention kernels of
libraries that ship with the image (library code: context for the reader, not a reference arm).
"""
import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOAD = "C2"
METRIC = "attention fwd+bwd TFLOP/s (BF16, causal)"
N_INPUT_SETS = 4          # rotated so a step never finds its inputs in L2 from the previous step


def flops(B, H, N, d, causal):
    pairs = B * H * N * N * (0.5 if causal else 1.0)
    return 4.0 * pairs * d, 10.0 * pairs * d


# dram__bytes_read.sum + dram__bytes_write.sum of one attn_bwd_kernel_d64 launch on C2 (ncu capture summarised in
# profiles/attn_bwd_kernel_d64_C2.md): 209.9 MB + 111.7 MB.
BWD_DRAM_BYTES_PER_LAUNCH_C2 = 321.7e6


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(bf16_tflops=float(p["bf16_tflops"]), hbm_gbs=float(p["hbm_gbs"]), source="measured")
    return dict(bf16_tflops=1590.0, hbm_gbs=6650.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed regions run."""

    def __init__(self, index):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _run(self):
        nv = self.nv
        names = {}
        for key, label in (("nvmlClocksEventReasonHwSlowdown", "hw_slowdown"),
                           ("nvmlClocksThrottleReasonHwSlowdown", "hw_slowdown"),
                           ("nvmlClocksEventReasonHwThermalSlowdown", "hw_thermal_slowdown"),
                           ("nvmlClocksThrottleReasonHwThermalSlowdown", "hw_thermal_slowdown"),
                           ("nvmlClocksEventReasonSwThermalSlowdown", "sw_thermal_slowdown"),
                           ("nvmlClocksThrottleReasonSwThermalSlowdown", "sw_thermal_slowdown"),
                           ("nvmlClocksEventReasonSwPowerCap", "sw_power_cap"),
                           ("nvmlClocksThrottleReasonSwPowerCap", "sw_power_cap")):
            if hasattr(nv, key):
                names[int(getattr(nv, key))] = label
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, label in names.items():
                    if r & bit:
                        self.reasons.add(label)
            except Exception:
                pass
            time.sleep(0.002)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return dict(sm_mhz=None, sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons), samples=0)
        s = sorted(self.samples)
        return dict(sm_mhz=s[len(s) // 2], sm_max_mhz=self.max_mhz, reasons=sorted(self.reasons),
                    samples=len(s))


def cpu_baseline(sample_heads, repeat=1, workload=WORKLOAD):
    """The oracle as it stands (BF16-emulating forward + delta + backward) timed on the host cores,
    on `sample_heads` heads of `workload`."""
    import attn_inputs as ai
    import oracle
    WORKLOAD = workload
    H0 = ai.CONFIGS[WORKLOAD][1]
    Bs, Hs = (sample_heads // H0, H0) if sample_heads % H0 == 0 else (1, sample_heads)
    t, m = ai.make(WORKLOAD, B=Bs, H=Hs)
    f_fwd, f_bwd = flops(Bs, Hs, m["N"], m["d"], m["causal"])
    best = None
    for _ in range(repeat):
        t0 = time.perf_counter()
        O, L = oracle.emu_fwd(t["q"], t["k"], t["v"], m["causal"], m["alpha"], 0)
        delta = oracle.emu_delta(O, t["dO"])
        oracle.emu_bwd(t["q"], t["k"], t["v"], t["dO"], L, delta, m["causal"], m["alpha"])
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    return dict(value=(f_fwd + f_bwd) / best / 1e12, unit="TFLOP/s", cores=oracle.num_threads(), kind="oracle",
                sample=f"BF16-emulating oracle fwd+delta+bwd on {sample_heads} of the "
                       f"{ai.CONFIGS[WORKLOAD][0] * ai.CONFIGS[WORKLOAD][1]} heads of {WORKLOAD} "
                       f"(B={Bs},H={Hs},N={m['N']},d={m['d']}), {best:.2f} s"), best


def run_reference(args):
    """Reference arm: the CPU oracle, timed as it stands on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import attn_inputs as ai
    heads = 2
    B0, H0, N, d, causal = ai.CONFIGS[WORKLOAD]
    for _ in range(args.warmup):
        cpu_baseline(heads)
    times = []
    base = None
    for _ in range(args.steps):
        base, dt = cpu_baseline(heads)
        times.append(dt)
    f_fwd, f_bwd = flops(1, heads, N, d, causal)
    total = sum(times)
    value = (f_fwd + f_bwd) * len(times) / total / 1e12
    base["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{WORKLOAD}: B={B0},H={H0},N={N},d={d},causal (sample of {heads} heads per step)"},
        "cpu_baseline": base,
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))



# heads of C4 / C5 the oracle is timed on (one head of either is 10-20 s of host work)
CPU_SAMPLE_HEADS = {"C4": 1, "C5": 1}


def other_workloads(attn, torch, steps=5, cpu=True):
    """Context lines for the other configurations of the scope table (the headline stays C2): device-timed
    fwd + bwd throughput with inputs resident in HBM, a few steps each.  Inputs are torch-seeded Gaussians of the
    configuration's shape (throughput does not depend on the values); C4 and C5 exceed the L2 by themselves,
    C2 in the stabilised mode rotates through input sets like the headline run."""
    import attn_inputs as ai
    out = {}
    for name, mode, nsets in (("C2", 1, N_INPUT_SETS), ("C4", 0, 1), ("C5", 0, 1)):
        B, H, N, d, causal = ai.CONFIGS[name]
        alpha = 1.0 / math.sqrt(d)
        gen = torch.Generator(device="cuda").manual_seed(1234)
        sets = []
        for _ in range(nsets):
            x = {n: torch.randn((B, H, N, d), device="cuda", generator=gen).to(torch.bfloat16) for n in ("q", "k", "v")}
            x["dO"] = (0.1 * torch.randn((B, H, N, d), device="cuda", generator=gen)).to(torch.bfloat16)
            sets.append(x)
        o = torch.empty_like(sets[0]["q"])
        lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
        delta = torch.empty_like(lse)
        dq, dk, dv = (torch.empty_like(o) for _ in range(3))
        ws_bytes = attn.attn_bwd_workspace_bytes(B, H, N, d)
        ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")

        def step(x):
            attn.attn_fwd(x["q"], x["k"], x["v"], o, lse, B, H, N, d, causal, alpha, mode)
            attn.attn_bwd(x["q"], x["k"], x["v"], o, x["dO"], lse, dq, dk, dv, delta, ws, ws_bytes,
                          B, H, N, d, causal, alpha, mode)

        for w in range(3):
            step(sets[w % nsets])
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(steps):
            step(sets[k % nsets])
        e1.record()
        torch.cuda.synchronize()
        if attn.attn_last_device_status() != 0:
            raise SystemExit("device-side wait timed out in " + name)
        ms = e0.elapsed_time(e1) / steps
        f_fwd, f_bwd = flops(B, H, N, d, causal)
        out[f"{name}_mode{mode}"] = {"shape": f"B={B},H={H},N={N},d={d},{'causal' if causal else 'full'}",
                                     "ms_per_step": ms, "tflops": (f_fwd + f_bwd) / (ms * 1e-3) / 1e12}
        del sets, o, lse, delta, dq, dk, dv, ws
        torch.cuda.empty_cache()
        if cpu and name in CPU_SAMPLE_HEADS:
            out[f"{name}_mode{mode}"]["cpu_baseline"], _ = cpu_baseline(CPU_SAMPLE_HEADS[name], workload=name)
    return out


def context_libs(torch, steps=20):
    """Library context (not a reference arm, no part of the product path): the headline workload's forward + backward
    through torch's scaled_dot_product_attention with its cuDNN and flash-attention back ends, on tensors of the same
    shape.  Each is captured into a CUDA graph (forward + autograd backward) and replayed, so that the time is the
    device's and not the host's; where capture fails the eager time is given and marked."""
    import attn_inputs as ai
    import torch.nn.functional as F
    from torch.nn.attention import SDPBackend, sdpa_kernel
    B, H, N, d, causal = ai.CONFIGS[WORKLOAD]
    f_fwd, f_bwd = flops(B, H, N, d, causal)
    gen = torch.Generator(device="cuda").manual_seed(99)
    sets = []
    for _ in range(N_INPUT_SETS):
        q, k, v = (torch.randn((B, H, N, d), device="cuda", generator=gen).to(torch.bfloat16).requires_grad_()
                   for _ in range(3))
        dO = (0.1 * torch.randn((B, H, N, d), device="cuda", generator=gen)).to(torch.bfloat16)
        sets.append((q, k, v, dO))
    out = {}
    for label, backend in (("torch_sdpa_cudnn", SDPBackend.CUDNN_ATTENTION), ("torch_sdpa_flash", SDPBackend.FLASH_ATTENTION)):
        try:
            with sdpa_kernel(backend):
                def one(x):
                    q, k, v, dO = x
                    o = F.scaled_dot_product_attention(q, k, v, is_causal=causal)
                    return torch.autograd.grad(o, (q, k, v), dO)

                for x in sets:
                    one(x)
                torch.cuda.synchronize()
                how = "cuda graph replay"
                try:
                    graphs = []
                    side = torch.cuda.Stream()
                    side.wait_stream(torch.cuda.current_stream())
                    with torch.cuda.stream(side):
                        for x in sets:
                            g = torch.cuda.CUDAGraph()
                            with torch.cuda.graph(g, stream=side):
                                keep = one(x)
                            graphs.append((g, keep))
                    torch.cuda.current_stream().wait_stream(side)
                    run = lambda i: graphs[i % len(graphs)][0].replay()
                except Exception:
                    torch.cuda.synchronize()
                    how = "eager (graph capture failed: host launch overhead included)"
                    run = lambda i: one(sets[i % len(sets)])
                for i in range(3):
                    run(i)
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for i in range(steps):
                    run(i)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1) / steps
                out[label] = {"ms_per_step": ms, "tflops": (f_fwd + f_bwd) / (ms * 1e-3) / 1e12, "how": how}
                # the forward alone (eager calls back to back: no autograd graph to build, the launches queue ahead)
                with torch.no_grad():
                    fwd_only = lambda i: F.scaled_dot_product_attention(*sets[i % len(sets)][:3], is_causal=causal)
                    for i in range(3):
                        fwd_only(i)
                    torch.cuda.synchronize()
                    e0.record()
                    for i in range(steps):
                        fwd_only(i)
                    e1.record()
                    torch.cuda.synchronize()
                out[label]["fwd_ms"] = e0.elapsed_time(e1) / steps
        except Exception as e:            # a back end that is not available for this shape on this machine
            out[label] = {"unavailable": str(e).splitlines()[0][:200]}
    return out

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--mode", type=int, default=0, choices=(0, 1))
    ap.add_argument("--impl", default="ours", choices=("ours", "reference"))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the context lines for C2 mode 1, C4 and C5")
    ap.add_argument("--scaling", default="weak", choices=("weak", "strong"),
                    help="weak: the whole batch on every rank; strong: one batch split over the ranks by (batch, head) ranges")
    ap.add_argument("--context-libs", action="store_true",
                    help="also time the image's library attention kernels on the same workload (context, printed under its own key)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import numpy as np
    import torch
    import attn_inputs as ai
    import paper_2510_04212_b200 as attn

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback for the hot path")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        # NCCL's own log (topology, NVLS, rings) is kept, in a file per rank so that stdout stays the one JSON line;
        # the only collectives here are the barrier and the MAX over ranks of the timings
        os.environ.setdefault("NCCL_DEBUG", "INFO")
        os.environ.setdefault("NCCL_DEBUG_FILE", "/tmp/nccl_bench_%h_%p.log")
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    B0, H0, N, d, causal = ai.CONFIGS[WORKLOAD]
    alpha = 1.0 / math.sqrt(d)
    mode = args.mode
    strong = args.scaling == "strong" and world > 1
    if strong:
        # one batch for the whole job: this rank owns a contiguous range of its (batch, head) problems and calls the
        # library on that range as a [1, heads, N, d] problem
        from paper_2510_04212_b200.sharding import head_slice, shard_view
        h0, h1 = head_slice(B0 * H0, world, rank)
        B, H = 1, h1 - h0
    else:
        B, H = B0, H0
    f_fwd, f_bwd = flops(B, H, N, d, causal)                 # this rank's share
    job_flops = sum(flops(B0, H0, N, d, causal)) * (1 if strong else world)

    # ---- inputs: N_INPUT_SETS seeded sets, resident in HBM before any timed region
    def dev_bf16(bits):
        return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).cuda().view(torch.bfloat16)

    host_sets, sets = [], []
    for s in range(N_INPUT_SETS):
        t, _ = ai.make(WORKLOAD, seed=ai.SEEDS[WORKLOAD] + 1000 * s + (0 if strong else 17 * rank))
        if strong:
            t = {n: shard_view(t[n], B0, H0, world, rank) for n in ("q", "k", "v", "dO")}
        host = {n: torch.from_numpy(np.ascontiguousarray(t[n]).view(np.int16)).view(torch.bfloat16).pin_memory()
                for n in ("q", "k", "v", "dO")}
        host_sets.append(host)
        sets.append({n: host[n].cuda() for n in host})
    o = torch.empty_like(sets[0]["q"])
    lse = torch.empty((B, H, N), dtype=torch.float32, device="cuda")
    delta = torch.empty_like(lse)
    dq, dk, dv = (torch.empty_like(o) for _ in range(3))
    ws_bytes = attn.attn_bwd_workspace_bytes(B, H, N, d)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda")

    def step(x):
        attn.attn_fwd(x["q"], x["k"], x["v"], o, lse, B, H, N, d, causal, alpha, mode)
        attn.attn_bwd(x["q"], x["k"], x["v"], o, x["dO"], lse, dq, dk, dv, delta, ws, ws_bytes,
                      B, H, N, d, causal, alpha, mode)

    def staged_step(x, ev):
        ev[0].record()
        attn.attn_fwd(x["q"], x["k"], x["v"], o, lse, B, H, N, d, causal, alpha, mode)
        ev[1].record()
        for st in (1, 2, 3):
            attn.attn_bwd_stage(st, x["q"], x["k"], x["v"], o, x["dO"], lse, dq, dk, dv, delta, ws, ws_bytes,
                                B, H, N, d, causal, alpha, mode)
            ev[1 + st].record()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for w in range(max(args.warmup, 3)):
        step(sets[w % N_INPUT_SETS])
    torch.cuda.synchronize()
    if attn.attn_last_device_status() != 0:
        raise SystemExit("device-side wait timed out during warm-up")

    with ClockSampler(local) as clocks:
        # ---- region A: K whole steps, device-timed
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for k in range(args.steps):
            step(sets[k % N_INPUT_SETS])
        e1.record()
        barrier()
        ms_total = e0.elapsed_time(e1)

        # ---- region A2: the same rotated steps, one event pair per step: the distribution of the step time (an event
        # between two steps keeps the next forward's prologue from overlapping the previous kernel's tail, so these
        # are a little longer than the mean of region A)
        n_each = max(20, args.steps)
        pe = [torch.cuda.Event(enable_timing=True) for _ in range(n_each + 1)]
        pe[0].record()
        for k in range(n_each):
            step(sets[k % N_INPUT_SETS])
            pe[k + 1].record()
        torch.cuda.synchronize()
        each = sorted(pe[k].elapsed_time(pe[k + 1]) for k in range(n_each))

        # ---- region A3: the same number of steps on ONE input set (its 101 MB of inputs and the outputs of the
        # previous step stay in the 126 MB L2 as far as they fit): the unflushed figure
        for w in range(3):
            step(sets[0])
        barrier()
        u0, u1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        u0.record()
        for k in range(args.steps):
            step(sets[0])
        u1.record()
        barrier()
        ms_single_set = u0.elapsed_time(u1) / args.steps

        # ---- region B: the same K steps with events between the kernels (per-kernel durations)
        evs = [[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(args.steps)]
        for k in range(args.steps):
            staged_step(sets[k % N_INPUT_SETS], evs[k])
        torch.cuda.synchronize()
        per_kernel = [sum(evs[k][i].elapsed_time(evs[k][i + 1]) for k in range(args.steps)) / args.steps
                      for i in range(4)]          # ms: fwd, preprocess, bwd main, dq convert

        # ---- region C: end to end from pinned host memory and back
        res_host = {n: torch.empty((B, H, N, d), dtype=torch.bfloat16).pin_memory() for n in ("o", "dq", "dk", "dv")}
        lse_host = torch.empty((B, H, N), dtype=torch.float32).pin_memory()
        stage_in = {n: torch.empty_like(sets[0][n]) for n in ("q", "k", "v", "dO")}
        e2e_steps = max(3, min(args.steps, 20))

        def e2e_step(hs):
            for n in stage_in:
                stage_in[n].copy_(hs[n], non_blocking=True)
            step(stage_in)
            res_host["o"].copy_(o, non_blocking=True)
            res_host["dq"].copy_(dq, non_blocking=True)
            res_host["dk"].copy_(dk, non_blocking=True)
            res_host["dv"].copy_(dv, non_blocking=True)
            lse_host.copy_(lse, non_blocking=True)

        e2e_step(host_sets[0])
        barrier()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for k in range(e2e_steps):
            e2e_step(host_sets[k % N_INPUT_SETS])
        c1.record()
        barrier()
        ms_e2e_serial = c0.elapsed_time(c1) / e2e_steps

        # The same steps as a pipeline: the host-to-device copy of step k+1 runs on a copy stream while step k's
        # results go back on another (the link is full duplex); inputs are staged in two device buffers, and step k+1
        # writes the other of two result sets while the results of step k leave.  Every step still copies
        # its inputs in from pinned host memory and all its results out, inside the timed region.
        cur = torch.cuda.current_stream()
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()
        stage2 = [stage_in, {n: torch.empty_like(stage_in[n]) for n in stage_in}]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        # two sets of result tensors as well, so that step k+1 computes while the results of step k travel
        outs2 = [dict(o=o, lse=lse, dq=dq, dk=dk, dv=dv),
                 dict(o=torch.empty_like(o), lse=torch.empty_like(lse), dq=torch.empty_like(dq),
                      dk=torch.empty_like(dk), dv=torch.empty_like(dv))]

        def step_into(x, r):
            attn.attn_fwd(x["q"], x["k"], x["v"], r["o"], r["lse"], B, H, N, d, causal, alpha, mode)
            attn.attn_bwd(x["q"], x["k"], x["v"], r["o"], x["dO"], r["lse"], r["dq"], r["dk"], r["dv"], delta, ws,
                          ws_bytes, B, H, N, d, causal, alpha, mode)

        def e2e_pipeline(steps, first, last):
            first.record(cur)
            for k in range(steps):
                b = k & 1
                with torch.cuda.stream(s_in):
                    if k == 0:
                        s_in.wait_event(first)
                    if k >= 2:
                        s_in.wait_event(ev_cmp[b])             # step k-2 has read this staging set
                    for n in stage2[b]:
                        stage2[b][n].copy_(host_sets[k % N_INPUT_SETS][n], non_blocking=True)
                    ev_in[b].record(s_in)
                cur.wait_event(ev_in[b])
                if k >= 2:
                    cur.wait_event(ev_out[b])                  # the results of step k-2 (same result set) have been copied out
                step_into(stage2[b], outs2[b])
                ev_cmp[b].record(cur)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_cmp[b])
                    res_host["o"].copy_(outs2[b]["o"], non_blocking=True)
                    res_host["dq"].copy_(outs2[b]["dq"], non_blocking=True)
                    res_host["dk"].copy_(outs2[b]["dk"], non_blocking=True)
                    res_host["dv"].copy_(outs2[b]["dv"], non_blocking=True)
                    lse_host.copy_(outs2[b]["lse"], non_blocking=True)
                    ev_out[b].record(s_out)
            last.record(s_out)

        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_pipeline(2, w0, w1)                                # warm-up
        barrier()
        p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e2e_pipeline(e2e_steps, p0, p1)
        barrier()
        ms_e2e = p0.elapsed_time(p1) / e2e_steps
    if attn.attn_last_device_status() != 0:
        raise SystemExit("device-side wait timed out during the timed region")

    ms_median = each[len(each) // 2]
    if dist is not None:
        tt = torch.tensor([ms_total, ms_e2e, ms_median, ms_single_set], device="cuda", dtype=torch.float64)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        ms_total, ms_e2e, ms_median, ms_single_set = (float(x) for x in tt)
    ms_step = ms_total / args.steps
    value = job_flops / (ms_step * 1e-3) / 1e12
    e2e_value = job_flops / (ms_e2e * 1e-3) / 1e12
    elem_bytes = B * H * N * d * 2

    if rank == 0:
        peaks = measured_peaks()
        bwd_ms = per_kernel[2]
        achieved = f_bwd / (bwd_ms * 1e-3) / 1e12
        clk = clocks.summary()
        # forward at d = 64: the exponentials bind before the tensor pipe does.  One ex2 per score pair that counts
        # (Pi = B*H*N^2/2), against 16 ex2 per clock per SM (4 per SM sub-partition) x 148 SMs x the SM clock
        # sampled during the timed regions.
        sm_mhz = clk["sm_mhz"] or clk["sm_max_mhz"] or 1965
        pairs = B * H * N * N * (0.5 if causal else 1.0)
        mufu_peak = 16 * 148 * sm_mhz * 1e6 / 1e9            # Gex2/s
        mufu_achieved = pairs / (per_kernel[0] * 1e-3) / 1e9
        out = {
            "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "strong" if strong else "weak",
            "ms_per_step_each": {"n": len(each), "median": ms_median, "min": each[0], "p90": each[(9 * len(each)) // 10],
                                 "max": each[-1], "how": "one CUDA-event pair per step, rotated input sets"},
            "ms_per_step_single_set": ms_single_set,
            "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": (f"{WORKLOAD}: B={B0},H={H0},N={N},d={d},causal, mode={mode} "
                                    + (f"(one batch split over {world} GPUs, {H} of {B0 * H0} heads on rank 0)" if strong
                                       else "(per GPU)")),
                       "l2": f"{N_INPUT_SETS} input sets rotated ({N_INPUT_SETS * 4 * elem_bytes / 1e6:.0f} MB > 126 MB L2)",
                       "flop_convention": "fwd 4*Pi*d + bwd 10*Pi*d, Pi=B*H*N^2/2"},
            "frac_of_bf16_peak": value / world / peaks["bf16_tflops"],
            "frac_of_nominal_2250": value / world / 2250.0,
            "frac_of_bf16_peak_median_step": (f_fwd + f_bwd) / (ms_median * 1e-3) / 1e12 / peaks["bf16_tflops"],
            "kernels_ms": {"attn_fwd_kernel": per_kernel[0], "bwd_preprocess_kernel": per_kernel[1],
                           "attn_bwd_kernel": per_kernel[2],
                           "dq_convert_tiled128_kernel": per_kernel[3] if d != 64 else None},
            "fwd_tflops": f_fwd / (per_kernel[0] * 1e-3) / 1e12,
            "delta_pass_gbs": (2 * elem_bytes + 4 * B * H * N) / (per_kernel[1] * 1e-3) / 1e9,
            "roofline_fwd": {"bound": "mufu", "kernel": "attn_fwd_kernel", "achieved": mufu_achieved, "peak": mufu_peak,
                             "unit": "Gex2/s", "frac": mufu_achieved / mufu_peak,
                             "peak_source": f"16 ex2/clk/SM x 148 SMs x {sm_mhz} MHz (median SM clock sampled in the timed regions)",
                             "tensor_frac": f_fwd / (per_kernel[0] * 1e-3) / 1e12 / peaks["bf16_tflops"]},
            "roofline": {"bound": "tensor", "kernel": "attn_bwd_kernel", "achieved": achieved,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                         "peak_source": peaks["source"] + " (burst)",
                         "traffic": BWD_DRAM_BYTES_PER_LAUNCH_C2 if (WORKLOAD == "C2" and not strong) else None,
                         "traffic_unit": "bytes per launch (ncu dram read + write, profiles/attn_bwd_kernel_d64_C2.md)"},
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": 4 * elem_bytes,
                    "d2h_bytes_per_step": 4 * elem_bytes + 4 * B * H * N, "ms_per_step": ms_e2e,
                    "how": "pipelined: H2D of step k+1 and D2H of step k on two copy streams around the compute stream, inputs and results double-buffered on the device",
                    "ms_per_step_serial": ms_e2e_serial},
            "gpu_launches": (3 if d == 64 else 4) * args.steps,   # d = 64: the main kernel also finishes dQ
            "clocks": clk,
        }
        if not args.no_cpu_baseline and world == 1:
            out["cpu_baseline"], _ = cpu_baseline(96)
        if world == 1 and not args.no_other_workloads:
            out["other_workloads"] = other_workloads(attn, torch, cpu=not args.no_cpu_baseline)
        if world == 1 and args.context_libs:
            out["context_libs"] = context_libs(torch)
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

"""Benchmark of the expert-choice MoE layer (forward + backward) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4|cfg2|small] [--impl reference]
  python bench.py --routing [--route-case n,E]      (routing-only stress, one extra JSON line format)
  python bench.py --sweep                           (capacity-factor sweep of the forward pass)

A step is one forward + backward pass of the whole layer over one group of n tokens
(routing, gather, expert FFNs, combine, and every backward kernel).  Prints ONE JSON
line.  `value` is tokens/s with all inputs resident in HBM; `e2e` is the same metric
with the step's inputs (X, dX_out) copied from pinned host memory and its results
(X_out, dX) copied back inside the timed region.  With N > 1 (torchrun) every rank
runs its own group on its own GPU: the layer routes each group independently, there
is no data-path collective, and the ranks are replicas (weak scaling).

`--impl reference` times the CPU oracle (fp64 numpy, as it stands) on the host cores
on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

WORKLOADS = {
    # name: (n, d, d', E, c)   shapes of Table 1 at sequence length 1024
    "cfg4": (16384, 4096, 16384, 64, 2.0),      # 8B/64E-shaped layer (headline)
    "cfg2": (8192, 768, 3072, 32, 2.0),         # 100M/32E-shaped layer
    "cfg4e4": (1024, 4096, 16384, 4, 2.0),      # four experts of the 8B/64E shape (profiling-sized)
    "cfg3c05": (8192, 768, 3072, 64, 0.5),      # capacity-factor sweep, 100M/64E shape: k = 64
    "cfg3c1": (8192, 768, 3072, 64, 1.0),       #   k = 128
    "cfg3c2": (8192, 768, 3072, 64, 2.0),       #   k = 256
    "small": (2048, 256, 512, 8, 2.0),
}
GEMM_STAGES = ("gemm1_gelu", "gemm2", "gemm_dZ", "gemm_dW2", "gemm_dW1", "gemm_dXin")


# nominal figures the targets are phrased against (context; the measured peaks are the roofline denominators)
NOMINAL_BF16_TFLOPS, NOMINAL_HBM_GBS = 2250.0, 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            j = json.load(f)
        return dict(hbm_gbs=j["hbm_gbs"], tflops_burst=j["bf16_tflops"],
                    tflops_sustained=j["bf16_tflops_sustained"], source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    INSTANT = None                      # whether this driver's nvidia-smi knows power.draw.instant (asked once)

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None
        if ClockSampler.INSTANT is None:
            try:
                ClockSampler.INSTANT = subprocess.run(["nvidia-smi", "--query-gpu=power.draw.instant", "--format=csv,noheader,nounits",
                                                       "-i", str(index)], capture_output=True, timeout=20).returncode == 0
            except Exception:
                ClockSampler.INSTANT = False

    def __enter__(self):
        try:
            q = self.Q + (",power.draw.instant" if ClockSampler.INSTANT else "")      # an eighth column: the unaveraged reading
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def __exit__(self, *a):
        if self.proc is not None:
            time.sleep(0.15)
            self.proc.terminate()
            self.thread.join(timeout=2)

    def summary(self):
        sm, mx, reasons = [], 0, set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx = max(mx, float(r[1]))
                for nme, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(nme)
            except Exception:
                pass
        sm.sort()
        def under_load(col):
            # samples taken under load: the sampler also sees the moments before the first and after the last launch
            w = []
            for r in self.rows:
                try:
                    w.append(float(r[col]))
                except Exception:
                    pass
            if not w:
                return None
            w = [x for x in w if x >= 0.8 * max(w)]
            return round(sum(w) / len(w), 1)
        # power.draw is the driver's running average (right for loops of seconds, low for a region of one second between
        # pauses); power.draw.instant is a snapshot (no lag, several percent of noise)
        watts, instant = under_load(2), under_load(7)
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": mx or None,
                "reasons": sorted(reasons), "samples": len(sm), "watts": watts, "watts_instant": instant}


def workload_desc(name, groups=1, cap_b=0, cap_iters=100, fuse_gather=False):
    n, d, dff, E, c = WORKLOADS[name]
    how = "one routing group per GPU" if groups == 1 else f"{groups} routing groups of {n // groups} tokens per GPU"
    if cap_b:
        how += f", at most {cap_b} experts per token ({cap_iters} solver rounds)"
    if fuse_gather:
        how += ", X_in read in place through I (fuse_gather)"
    return (f"{name}: n={n} d={d} d_ff={dff} E={E} c={c} k={int(n * c / E)} fwd+bwd, bf16 storage / fp32 accumulate, "
            f"{how}")


GEMM_PROFILE = os.path.join(ROOT, "profiles", "gemm_tc_kernel_cfg4e4.md")
GEMM_SOURCE = os.path.join(ROOT, "paper_2202_09368_b200", "csrc", "gemm_tc.cu")


def source_digest(path=GEMM_SOURCE):
    import hashlib
    with open(path, "rb") as f:
        return hashlib.sha256(f.read()).hexdigest()[:16]


def gemm_traffic(workload, E):
    """DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per expert-GEMM launch, mean over the six launches of
    a step, read from the ncu summary under profiles/ (a capture of four experts of the 8B/64E shape: operands,
    outputs and weights all grow with the number of experts, so a launch at E experts moves E/4 times as much).
    None for shapes that were not captured, and None when the kernel source is no longer the one that was captured
    (the summary records a digest of it)."""
    if workload not in ("cfg4", "cfg4e4") or not os.path.exists(GEMM_PROFILE):
        return None
    rd = wr = None
    digest = None
    for line in open(GEMM_PROFILE):
        cells = [c.strip() for c in line.split("|")]
        if len(cells) > 3 and cells[1] in ("dram__bytes_read.sum", "dram__bytes_write.sum") and cells[2] == "Mbyte":
            vals = [float(c) for c in cells[3:] if c]
            if cells[1].endswith("read.sum"):
                rd = vals
            else:
                wr = vals
        if line.startswith("kernel source digest:"):
            digest = line.split(":", 1)[1].strip().strip("`")
    if not rd or not wr or len(rd) != len(wr) or digest != source_digest():
        return None
    per_launch_e4 = sum(a + b for a, b in zip(rd, wr)) / len(rd) * 1e6          # the table is in Mbyte
    return per_launch_e4 * E / 4


def layer_flops(n, d, dff, E, c):
    slots = int(n * c)
    gemm = 2.0 * slots * d * dff                 # one expert-batched GEMM
    gate = 2.0 * n * d * E
    return dict(gemm=gemm, fwd=2 * gemm + gate, bwd=4 * gemm + 2 * gate)


# ----------------------------------------------------------------------------------- CPU oracle timing
def time_oracle_sample(n, d, dff, E, c, seed=0, budget_s=12.0, groups=1):
    """Times the oracle on routing in full plus as many whole experts forward + backward as fit in
    about `budget_s` seconds of CPU work (at least one, at most E) and extrapolates the expert part
    to E experts.  Returns (tokens/s, threads, description)."""
    import numpy as np
    import torch
    from oracle import ec_oracle as O
    from paper_2202_09368_b200 import inputs as IN
    try:
        from threadpoolctl import threadpool_info
        threads = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        threads = os.cpu_count() or 1
    bf = torch.bfloat16
    X = IN.normal_tensor((n, d), 1.0, seed, IN.TID_X, bf).float().numpy().astype(np.float64)
    Wg = IN.normal_tensor((d, E), 1.0 / math.sqrt(d), seed, IN.TID_WG, bf).float().numpy().astype(np.float64)
    dY = IN.normal_tensor((n, d), 1.0, seed, IN.TID_DXOUT, bf).float().numpy().astype(np.float64)
    per = d * dff

    def weights(tid, i, fan_in):
        w = (IN.normal_chunk(seed, tid, i * per, per) / math.sqrt(fan_in)).to(bf)
        return w.float().numpy().astype(np.float64).reshape(d, dff)

    t0 = time.perf_counter()
    r = O.route(X, Wg, c, groups=groups)
    t_route = time.perf_counter() - t0
    t_sum, experts = 0.0, 0
    k = r["I"].shape[1]
    X_out, dX = np.zeros((n, d)), np.zeros((n, d))
    dG = np.zeros((E, k))
    while experts < E and (experts == 0 or t_route + t_sum < budget_s):
        i = experts
        W1_i, W2_i = weights(IN.TID_W1, i, d), weights(IN.TID_W2, i, dff)      # generation is not timed
        t0 = time.perf_counter()
        I_i, G_i = r["I"][i:i + 1], r["G"][i:i + 1]
        X_in = X[I_i[0]]
        Z, H, X_e = O.expert_ffn(X_in, W1_i, W2_i)
        X_out += O.combine(X_e[None], G_i, I_i, n)                             # Eq. 4, this expert's share
        dX_e = G_i[0][:, None] * dY[I_i[0]]
        dG[i] = np.einsum("jd,jd->j", dY[I_i[0]], X_e)
        _, _, dX_in, _, _ = O.expert_ffn_backward(dX_e, X_in, Z, H, W1_i, W2_i)
        O.add_slot_rows(dX, I_i, dX_in[None])
        t_sum += time.perf_counter() - t0
        experts += 1
    t0 = time.perf_counter()                                                   # the gate's backward, in full
    _, dL = O.softmax_backward(r["S"], r["I"], dG)
    dWg = X.T @ dL
    dX += dL @ Wg.T
    t_gate = time.perf_counter() - t0
    t_exp = t_sum / experts
    total = t_route + E * t_exp + t_gate
    what = (f"oracle (numpy fp64) on n={n} d={d} d'={dff} E={E} c={c}: routing in full ({t_route:.2f} s) + "
            f"{experts} of {E} experts forward+backward with their share of the combine ({t_exp:.2f} s each), expert part "
            f"extrapolated x{E}; gate backward in full ({t_gate:.2f} s)")
    return n / total, threads, what


def run_reference(args):
    n, d, dff, E, c = WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # every step is a bounded sample of the workload (seconds of CPU work); at most two are run however many were asked for
    ran = max(1, min(args.steps, 2))
    vals = []
    for _ in range(ran):
        v, threads, what = time_oracle_sample(n, d, dff, E, c, groups=args.groups)
        vals.append(v)
    v = sum(vals) / len(vals)
    out = {"impl": "reference", "metric": "ec_moe_layer_tokens_per_s_fwd_bwd", "value": v, "unit": "tokens/s",
           "n_gpus": args.gpus, "steps": ran, "steps_requested": args.steps, "warmup": 0, "ms_per_step": 1e3 * n / v,
           "ms_per_step_is": "extrapolated: the time of one whole step at the sampled rate, not the time the sample took",
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": workload_desc(args.workload, args.groups, args.cap_b, args.cap_iters, args.fuse_gather)},
           "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": what},
           "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


# ----------------------------------------------------------------------------------- GPU arm
def aggregate_max(t_local_ms: float, device) -> float:
    """Max over ranks of a per-rank time (one all-reduce on the bench's process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()):
        return t_local_ms
    t = torch.tensor([t_local_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2202_09368_b200 import binding as B
    from paper_2202_09368_b200 import inputs as IN

    rank = int(os.environ.get("RANK", "0")); world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    n, d, dff, E, c = WORKLOADS[args.workload]
    bf = torch.bfloat16
    assert n % args.groups == 0
    cfg = B.make_config(n // args.groups, d, dff, E, c, bf, groups=args.groups, cap_b=args.cap_b, cap_iters=args.cap_iters,
                        fuse_gather=args.fuse_gather)
    seed = rank                                                   # each rank routes its own group
    chunk = 1 << 26
    X = IN.normal_tensor((n, d), 1.0, seed, IN.TID_X, bf, dev, chunk)
    Wg = IN.normal_tensor((d, E), 1.0 / math.sqrt(d), seed, IN.TID_WG, bf, dev, chunk)
    W1 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(d), seed, IN.TID_W1, bf, dev, chunk)
    W2 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(dff), seed, IN.TID_W2, bf, dev, chunk)
    dY = IN.normal_tensor((n, d), 1.0, seed, IN.TID_DXOUT, bf, dev, chunk)
    ws = B.alloc_workspace(cfg, dev); saved = B.alloc_saved(cfg, dev)
    X_out = torch.empty_like(X)
    grads = (torch.empty_like(X), torch.empty_like(Wg), torch.empty_like(W1), torch.empty_like(W2))

    def step():
        B.ec_moe_forward(cfg, X, Wg, W1, W2, X_out, saved, ws)
        B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, grads, ws)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    assert B.ec_read_status(ws) == B.EC_OK
    if args.graph:
        # the step as one CUDA graph: the library only queues work on the given stream, so a forward + backward
        # pair can be captured once and replayed, which takes the launch latencies out of small steps
        side = torch.cuda.Stream(dev)
        side.wait_stream(torch.cuda.current_stream(dev))
        with torch.cuda.stream(side):
            step()
        torch.cuda.current_stream(dev).wait_stream(side)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        eager_step, step = step, graph.replay
        step(); torch.cuda.synchronize()
    # ---- timed region: K steps, device timed, max over ranks; repeated R times in this run so that the line can say
    # how much one region differs from the next on this machine (the SM clock under the power cap moves by several
    # percent).  `value` is the median region; the clock sampled during each region is reported beside its time.
    repeats = max(1, args.repeats)
    region_ms, region_mhz, launches, all_rows = [], [], 0, []
    for rep in range(repeats):
        barrier()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        l0 = B.ec_launch_count()
        with ClockSampler(local) as clocks:
            ev0.record()
            for _ in range(args.steps):
                step()
            ev1.record()
            barrier()
        launches = B.ec_launch_count() - l0
        region_ms.append(aggregate_max(ev0.elapsed_time(ev1), dev) / args.steps)
        region_mhz.append(clocks.summary()["sm_mhz"])
        all_rows += clocks.rows
    clocks.rows = all_rows                                         # the summary on the line covers every region
    order = sorted(range(repeats), key=lambda i: region_ms[i])
    ms_step = region_ms[order[repeats // 2]]
    assert B.ec_read_status(ws) == B.EC_OK

    # ---- per-stage times (CUDA events recorded by the library on the launching stream).  Steps are
    # queued back to back, as in the timed region, and only the last step of each burst is read, so
    # the stages are timed in the same sustained (power-capped) state as `value`.
    B.ec_profile_enable(True)
    stage_ms = {}
    bursts, burst_steps = 6, max(2, min(args.steps, 10))
    plain_step = eager_step if args.graph else step         # the stage events are recorded at launch time
    for _ in range(bursts):
        for _ in range(burst_steps):
            plain_step()
        for k_, v_ in B.ec_profile_read():
            stage_ms[k_] = stage_ms.get(k_, 0.0) + v_ / bursts
    B.ec_profile_enable(False)

    # ---- end to end: host buffers in, host buffers out, every copy inside the timed region.  Each step's X and
    # dX_out come from pinned host memory and its X_out and dX go back to pinned host memory; device input and
    # output buffers are double-buffered and the copies run on streams of their own, so the copy engines work on
    # step i+1's inputs and step i-1's results while step i computes.  Time is taken on the compute stream's
    # clock from before the first copy is queued until the last result has landed.
    hX, hdY = X.cpu().pin_memory(), dY.cpu().pin_memory()
    hOut, hdX = torch.empty_like(hX).pin_memory(), torch.empty_like(hX).pin_memory()
    s_in, s_out, s_cmp = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.current_stream(dev)
    bufs = [dict(X=torch.empty_like(X), dY=torch.empty_like(dY), X_out=torch.empty_like(X), dX=torch.empty_like(X),
                 loaded=torch.cuda.Event(), computed=torch.cuda.Event(), drained=torch.cuda.Event()) for _ in range(2)]

    def e2e_run(count):
        for i in range(count):
            b = bufs[i & 1]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(b["computed"])            # step i-2 has finished reading this pair of inputs
                b["X"].copy_(hX, non_blocking=True); b["dY"].copy_(hdY, non_blocking=True)
                b["loaded"].record(s_in)
            s_cmp.wait_event(b["loaded"])
            if i >= 2:
                s_cmp.wait_event(b["drained"])                # step i-2's results have left this pair of outputs
            B.ec_moe_forward(cfg, b["X"], Wg, W1, W2, b["X_out"], saved, ws)
            B.ec_moe_backward(cfg, b["X"], Wg, W1, W2, b["dY"], saved, (b["dX"],) + tuple(grads[1:]), ws)
            b["computed"].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(b["computed"])
                hOut.copy_(b["X_out"], non_blocking=True); hdX.copy_(b["dX"], non_blocking=True)
                b["drained"].record(s_out)
        s_cmp.wait_stream(s_out)                               # the last results are on the host

    e2e_run(2)
    barrier()
    e_steps = max(2, min(args.steps, 10))
    ev0.record()
    e2e_run(e_steps)
    ev1.record()
    barrier()
    e2e_ms = aggregate_max(ev0.elapsed_time(ev1), dev) / e_steps
    assert torch.equal(hOut, X_out.cpu()) and torch.equal(hdX, grads[0].cpu())     # same bits as the resident run
    io_bytes = X.numel() * 2 * 2

    fl = layer_flops(n, d, dff, E, c)
    peaks = measured_peaks()
    gemm_ms = [stage_ms[s] for s in GEMM_STAGES if s in stage_ms]
    gemm_avg_ms = sum(gemm_ms) / max(1, len(gemm_ms))
    achieved = fl["gemm"] / (gemm_avg_ms * 1e-3) / 1e12 if gemm_ms else None
    peak = peaks["tflops_sustained"]
    # This box's own sustained matmul rate, taken after all timed work with the vendor library (an 8192-cubed bf16 product in
    # a loop of about a second and a half, the kind of loop the pool's peak figure comes from).  Context for the fraction
    # above: the boxes of the pool differ by more than ten percent under the same power cap.  Calibration only.
    box_peak = None
    if world == 1 and args.workload == "cfg4" and not args.graph:
        a8, b8, c8 = (torch.randn(8192, 8192, device=dev, dtype=bf) for _ in range(3))
        for _ in range(20):
            torch.mm(a8, b8, out=c8)
        q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize(); q0.record()
        for _ in range(1800):
            torch.mm(a8, b8, out=c8)
        q1.record(); torch.cuda.synchronize()
        box_peak = 1800 * 2.0 * 8192 ** 3 / (q0.elapsed_time(q1) * 1e-3) / 1e12
        del a8, b8, c8

    if rank == 0:
        cpu = None
        if world == 1 and not args.no_cpu_baseline:
            v, threads, what = time_oracle_sample(n, d, dff, E, c, groups=args.groups)
            cpu = {"value": v, "unit": "tokens/s", "cores": threads, "kind": "oracle", "sample": what}
        out = {
            "metric": "ec_moe_layer_tokens_per_s_fwd_bwd", "value": world * n / (ms_step * 1e-3), "unit": "tokens/s",
            "n_gpus": world, "steps": args.steps, "warmup": max(3, args.warmup), "ms_per_step": ms_step,
            "regions": {"count": repeats, "steps_each": args.steps, "ms_per_step": [round(v, 4) for v in region_ms],
                        "sm_mhz": region_mhz, "median_ms": round(ms_step, 4), "best_ms": round(min(region_ms), 4),
                        "ms_x_mhz": [round(a * b, 1) if b else None for a, b in zip(region_ms, region_mhz)]},
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": workload_desc(args.workload, args.groups, args.cap_b, args.cap_iters, args.fuse_gather),
                       "l2": "inputs larger than L2 (weights + activations per step >> 126 MB), no flush"
                             if args.workload != "small" else "small case, L2 resident",
                       "tensor_cores": bool(B.ec_uses_tensor_cores(cfg)),
                       "launch": "one CUDA graph per step" if args.graph else "stream launches"},
            "clocks": clocks.summary(),
            "e2e": {"value": world * n / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": io_bytes,
                    "d2h_bytes_per_step": io_bytes, "ms_per_step": e2e_ms},
            "gpu_launches": launches,
            "roofline": {"bound": "tensor", "kernel": "gemm_tc_kernel (6 launches per step: the expert GEMMs of Eq. 3 "
                                                      "and their backward)",
                         "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": (achieved / peak) if achieved else None,
                         "frac_of_nominal": (achieved / NOMINAL_BF16_TFLOPS) if achieved else None,
                         "box_matmul_tflops": box_peak, "frac_of_box_matmul": (achieved / box_peak) if achieved and box_peak else None,
                         "peak_source": f"{peaks['source']} bf16 matmul, sustained", "traffic": gemm_traffic(args.workload, E),
                         "flops_per_launch": fl["gemm"], "avg_launch_ms": gemm_avg_ms},
            "stage_ms": {k_: round(v_, 4) for k_, v_ in stage_ms.items()},
            "saved_bytes": int(B.ec_saved_bytes(cfg)),
            "layer_tflops": (fl["fwd"] + fl["bwd"]) / (ms_step * 1e-3) / 1e12,
            # under the board's power cap a step costs what it costs in energy: watts (mean of the samples taken
            # under load; the unaveraged reading where nvidia-smi has one, a timed region being too short for the averaged one) x time per step; per flop of the layer it compares with the vendor's large square product
            # (`--gemms --loop-seconds`)
            "energy": (lambda c: (lambda w: {"watts": w, "source": "power.draw.instant" if c["watts_instant"] else "power.draw",
                                             "joules_per_step": round(w * ms_step * 1e-3, 3),
                                             "pj_per_flop": round(w * ms_step * 1e-3 / (fl["fwd"] + fl["bwd"]) * 1e12, 4)} if w else None)
                       (c["watts_instant"] or c["watts"]))(clocks.summary()),
            "cpu_baseline": cpu,
        }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------- routing-only stress
ROUTING_GRID = [(n, E) for n in (4096, 16384, 65536, 262144) for E in (8, 32, 128, 256)]


def routing_bytes(n, d, E, c, b=2, cap_iters=0):
    """Algorithmic bytes each routing stage has to move (reads + writes), per call.  The capped solver reads and
    writes log A and the box factors (fp32) once per round; that state stays in L2 at these sizes."""
    slots = int(n * c)
    return {
        "capped_assignment": cap_iters * 4 * n * E * 4 + 2 * n * E * 4,
        "gate_softmax": n * d * b + d * E * b + n * E * 4,
        "topk": n * E * 4 + slots * 8,
        "inverse_index": slots * 4 + (n + 1 + slots) * 4,
        "gather": 2 * slots * d * b + slots * 4,
        "combine": slots * d * 4 + slots * 4 + (n + 1 + slots) * 4 + n * d * b,
    }


def run_routing(args):
    """Routing-only stress: gate + softmax, column top-k, inverse index, shuffle and unshuffle with
    identity experts (X_e = X_in), d = 1024, bf16, c = 2.  Per stage: device time from the library's
    stage events and algorithmic GB/s.  L2 is flushed (a 512 MiB buffer is overwritten) before every
    timed call, so the small cases are not timed out of cache."""
    import torch
    from paper_2202_09368_b200 import binding as B
    from paper_2202_09368_b200 import inputs as IN
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    dev = torch.device("cuda")
    d, c, bf = 1024, 2.0, torch.bfloat16
    grid = ROUTING_GRID
    if args.route_case:                                   # "n,E" or "n,E,d"
        vals = [int(v) for v in args.route_case.split(",")]
        grid = [tuple(vals[:2])]
        d = vals[2] if len(vals) > 2 else d
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    peaks = measured_peaks()
    cases = []
    B.ec_profile_enable(True)
    for n, E in grid:
        cfg = B.make_config(n, d, 8, E, c, bf, cap_b=args.cap_b, cap_iters=args.cap_iters)
        X = IN.normal_tensor((n, d), 1.0, 0, IN.TID_X, bf, dev, 1 << 26)
        Wg = IN.normal_tensor((d, E), 1.0 / math.sqrt(d), 0, IN.TID_WG, bf, dev, 1 << 26)
        ws = B.alloc_workspace(cfg, dev)
        r = B.ec_route(cfg, X, Wg, ws=ws)
        X_in = B.ec_shuffle(cfg, X, r.I)
        X_e = X_in.float()
        X_out = torch.empty_like(X)
        acc = {}
        reps = max(3, min(args.steps, 20))
        for it in range(3 + reps):
            for call in (lambda: B.ec_route(cfg, X, Wg, ws=ws, out=r), lambda: B.ec_shuffle(cfg, X, r.I, X_in),
                         lambda: B.ec_unshuffle(cfg, X_e, r.G, r.row_ptr, r.slots, X_out)):
                flush.zero_()
                call()
                for k_, v_ in B.ec_profile_read():
                    if it >= 3:
                        acc.setdefault(k_, []).append(v_)
        assert B.ec_read_status(ws) == B.EC_OK
        # no case is printed whose output has not passed the checks that hold at any size (the parity tests compare
        # these sizes with the oracle element by element; here: properties, on the device, with torch)
        k = B.ec_capacity(cfg)
        assert B.ec_validate_routing(cfg, r.I, r.row_ptr, r.slots, ws) == 0, "inconsistent index structure"
        assert int(r.row_ptr[-1]) == E * k
        cols = torch.arange(E, device=dev).unsqueeze(1).expand(E, k)
        if not args.cap_b:
            assert torch.equal(r.G, r.S[r.I.long(), cols]), "G is not S at the selected pairs"
            chosen = torch.zeros(n, E, dtype=torch.bool, device=dev)
            chosen[r.I.long(), cols] = True
            assert int(chosen.sum()) == E * k, "an expert holds a token twice"
            lowest_in = torch.where(chosen, r.S, torch.full_like(r.S, 2.0)).amin(dim=0)
            highest_out = torch.where(chosen, torch.full_like(r.S, -1.0), r.S).amax(dim=0)
            assert bool((lowest_in >= highest_out).all()), "a token outside an expert's top k scores higher than one inside"
            assert bool((r.G[:, :-1] >= r.G[:, 1:]).all()), "an expert's slots are not in descending score order"
            del chosen, lowest_in, highest_out
        assert torch.equal(X_in, X[r.I.long()]), "the shuffle is not a copy of the selected rows"
        by = routing_bytes(n, d, E, c, cap_iters=args.cap_iters if args.cap_b else 0)
        st = {}
        for k_, v_ in acc.items():
            v_.sort()
            med = v_[len(v_) // 2]
            st[k_] = {"us": round(med * 1e3, 2), "GBps": round(by[k_] / (med * 1e-3) / 1e9, 1),
                      "frac_hbm": round(by[k_] / (med * 1e-3) / 1e9 / peaks["hbm_gbs"], 3),
                      "frac_nominal": round(by[k_] / (med * 1e-3) / 1e9 / NOMINAL_HBM_GBS, 3)}
        total_us = sum(v["us"] for v in st.values())
        cases.append({"n": n, "E": E, "d": d, "k": int(n * c / E), "stages": st, "chain_us": round(total_us, 2),
                      "chain_GBps": round(sum(by[k_] for k_ in st) / (total_us * 1e-6) / 1e9, 1),
                      "tokens_per_s": round(n / (total_us * 1e-6))})
        if args.cap_b:                                    # what the cap did to the number of experts per token
            cases[-1]["cap"] = {"b": args.cap_b, "rounds": args.cap_iters, "lambda": 1e-3,
                                "experts_per_token_hist": torch.bincount(r.row_ptr[1:] - r.row_ptr[:-1]).tolist()}
        del X, Wg, ws, r, X_in, X_e, X_out
    B.ec_profile_enable(False)
    print(json.dumps({"metric": "ec_routing_chain", "unit": "GB/s (algorithmic bytes / device time per stage)",
                      "config": {"workload": "routing-only stress: d=1024 bf16 c=2, identity experts",
                                 "l2": "512 MiB flush before every timed call",
                                 "checked": "every case: status word, ec_validate_routing, G = S at I, k distinct tokens per expert, "
                                            "threshold and order of every expert's scores, shuffle = row copy"},
                      "hbm_peak_gbs": peaks["hbm_gbs"], "peak_source": peaks["source"], "cases": cases}))


# ----------------------------------------------------------------------------------- capacity-factor sweep
def run_sweep(args):
    """Forward pass of the 100M/64E-shaped layer (n=8192, d=768, d'=3072, E=64, bf16) for c in {0.5, 1, 2} and gate
    logits scaled x1 and x4 (the scale multiplies Wg and varies how unevenly tokens are scored).  Per case: forward
    time (forward-only call, Z not stored), per-stage times, the expert GEMMs against both rooflines (with k = 64 to
    256 rows per expert they are bound by reading the 302 MB of W1 or W2, not by the tensor cores), and the histogram
    of the number of experts per token that the routing produced (the quantity of the paper's Fig. 3)."""
    import torch
    from paper_2202_09368_b200 import binding as B
    from paper_2202_09368_b200 import inputs as IN
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    dev = torch.device("cuda")
    n, d, dff, E, bf = 8192, 768, 3072, 64, torch.bfloat16
    peaks = measured_peaks()
    X = IN.normal_tensor((n, d), 1.0, 0, IN.TID_X, bf, dev, 1 << 26)
    W1 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(d), 0, IN.TID_W1, bf, dev, 1 << 26)
    W2 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(dff), 0, IN.TID_W2, bf, dev, 1 << 26)
    Y = torch.empty_like(X)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    cases = []
    for scale in (1.0, 4.0):
        Wg = IN.normal_tensor((d, E), scale / math.sqrt(d), 0, IN.TID_WG, bf, dev, 1 << 26)
        for c in (0.5, 1.0, 2.0):
            cfg = B.make_config(n, d, dff, E, c, bf)
            ws = torch.empty(int(B.lib().ec_forward_only_workspace_bytes(__import__("ctypes").byref(cfg))), dtype=torch.uint8, device=dev)
            reps = max(5, min(args.steps, 30))
            for _ in range(3):
                B.ec_moe_forward(cfg, X, Wg, W1, W2, Y, None, ws, forward_only=True)
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
            B.ec_profile_enable(True)
            acc = {}
            for a, b_ in ev:
                flush.zero_()                                   # the weights (604 MB) exceed L2 anyway; the activations do not
                a.record()
                B.ec_moe_forward(cfg, X, Wg, W1, W2, Y, None, ws, forward_only=True)
                b_.record()
                for k_, v_ in B.ec_profile_read():
                    acc.setdefault(k_, []).append(v_)
            B.ec_profile_enable(False)
            torch.cuda.synchronize()
            ms = sorted(a.elapsed_time(b_) for a, b_ in ev)[reps // 2]
            st = {k_: round(sorted(v_)[len(v_) // 2], 4) for k_, v_ in acc.items()}
            r = B.ec_route(cfg, X, Wg)
            per_token = (r.row_ptr[1:] - r.row_ptr[:-1]).long()
            hist = torch.bincount(per_token, minlength=1).tolist()
            k = int(n * c / E)
            flops = 2.0 * n * c * d * dff                       # one expert GEMM
            wbytes = E * d * dff * 2
            gem = {}
            for g_ in ("gemm1_gelu", "gemm2"):
                t = st[g_] * 1e-3
                gem[g_] = {"ms": st[g_], "TFLOPs": round(flops / t / 1e12, 1), "frac_tensor": round(flops / t / 1e12 / peaks["tflops_burst"], 3),
                           "weight_GBps": round(wbytes / t / 1e9, 1), "frac_hbm": round(wbytes / t / 1e9 / peaks["hbm_gbs"], 3)}
            cases.append({"c": c, "logit_scale": scale, "k": k, "forward_ms": round(ms, 4), "tokens_per_s": round(n / (ms * 1e-3)),
                          "stage_ms": st, "expert_gemms": gem, "experts_per_token_hist": hist,
                          "tokens_without_expert": hist[0], "max_experts_per_token": len(hist) - 1})
    print(json.dumps({"metric": "ec_moe_forward_capacity_sweep", "unit": "ms (median, forward only)",
                      "config": {"workload": f"capacity-factor sweep: n={n} d={d} d_ff={dff} E={E} bf16 forward, c x logit scale",
                                 "l2": "512 MiB flush before every timed call"},
                      "peaks": {"hbm_gbs": peaks["hbm_gbs"], "bf16_tflops_burst": peaks["tflops_burst"], "source": peaks["source"]},
                      "cases": cases}))


# ----------------------------------------------------------------------------------- expert GEMMs alone
def run_gemms(args):
    """The three expert-batched products of the layer, each alone in a loop (ec_expert_gemm), and torch.bmm (the vendor
    library) on the same buffers beside them, alternating, for calibration: what the tensor cores give this shape when
    nothing else runs.  16 experts of the workload's shape (the weight gradients then write 2 GiB per call at 8B/64E)."""
    import torch
    from paper_2202_09368_b200 import binding as B
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    dev, bf = torch.device("cuda"), torch.bfloat16
    n, d, dff, E, c = WORKLOADS[args.workload]
    Eb = min(E, 16)
    cfg = B.make_config(n * Eb // E, d, dff, Eb, c, bf)
    k = B.ec_capacity(cfg)
    A = torch.randn(Eb, k, d, device=dev, dtype=bf)
    H = torch.randn(Eb, k, dff, device=dev, dtype=bf)
    W = torch.randn(Eb, d, dff, device=dev, dtype=bf) * 0.02
    ws = B.alloc_workspace(cfg, dev)
    outs = {B.EC_GEMM_XW1: torch.empty(Eb, k, dff, device=dev, dtype=bf), B.EC_GEMM_HW2T: torch.empty(Eb, k, d, device=dev, dtype=bf),
            B.EC_GEMM_ATB: torch.empty(Eb, d, dff, device=dev, dtype=bf)}
    flops = 2.0 * Eb * k * d * dff
    cases = [("Z = X_in . W1", B.EC_GEMM_XW1, A, W, lambda o: torch.bmm(A, W, out=o)),
             ("X_e = H . W2^T", B.EC_GEMM_HW2T, H, W, lambda o: torch.bmm(H, W.transpose(1, 2), out=o)),
             ("dW = A^T . B", B.EC_GEMM_ATB, A, H, lambda o: torch.bmm(A.transpose(1, 2), H, out=o))]
    reps = max(10, args.steps)
    res = {}

    def timed(fn, count):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(count):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / count

    if args.loop_seconds > 0:
        # Energy view: every product loops for --loop-seconds, long enough for the power controller to settle and for
        # nvidia-smi to sample power and clocks; energy per flop = mean watts under load x time per call / flops.  A large square
        # product of the vendor library (nothing but tensor-core work, hardly any HBM traffic) calibrates the scale.
        side = 8192
        Sa, Sb, Sc = (torch.randn(side, side, device=dev, dtype=bf) for _ in range(3))
        loops = [("square 8192^3", "torch_mm", lambda: torch.mm(Sa, Sb, out=Sc), 2.0 * side ** 3)]
        for name, kind, a, b_, vendor in cases:
            loops.append((name, "this_library", (lambda kind=kind, a=a, b_=b_: B.ec_expert_gemm(cfg, kind, a, b_, outs[kind], ws)), flops))
            loops.append((name, "torch_bmm", (lambda kind=kind, vendor=vendor: vendor(outs[kind])), flops))
        for name, tag, fn, fl in loops:
            for _ in range(5):
                fn()
            count = max(20, int(args.loop_seconds * 1e3 / timed(fn, 10)))
            with ClockSampler(torch.cuda.current_device()) as cs:
                ms = timed(fn, count)
            c = cs.summary()
            res.setdefault(name, {})[tag] = {"tflops": round(fl / ms / 1e9, 1), "ms": round(ms, 4), "sm_mhz": c["sm_mhz"], "watts": c["watts"], "watts_instant": c["watts_instant"],
                                             "pj_per_flop": round(c["watts"] * ms * 1e-3 / fl * 1e12, 4) if c["watts"] else None,
                                             "reasons": c["reasons"]}
            time.sleep(0.5)
        assert B.ec_read_status(ws) == B.EC_OK
        print(json.dumps({"metric": "expert_gemm_alone_energy", "unit": "each product alone in a loop of --loop-seconds; pJ per flop = watts x time / flops",
                          "config": {"workload": f"{Eb} experts of {args.workload}: k={k} d={d} d_ff={dff}, bf16", "loop_seconds": args.loop_seconds},
                          "cases": res}))
        return
    for rnd in range(max(2, min(args.repeats, 3))):
        for name, kind, a, b_, vendor in cases:
            o = outs[kind]
            for tag, fn in (("this_library", lambda: B.ec_expert_gemm(cfg, kind, a, b_, o, ws)), ("torch_bmm", lambda: vendor(o))):
                for _ in range(5):
                    fn()
                res.setdefault(name, {}).setdefault(tag, []).append(round(flops / timed(fn, reps) / 1e9, 1))
    assert B.ec_read_status(ws) == B.EC_OK
    print(json.dumps({"metric": "expert_gemm_alone_tflops", "unit": "TFLOP/s, each product alone in a loop, rounds in order",
                      "config": {"workload": f"{Eb} experts of {args.workload}: k={k} d={d} d_ff={dff}, bf16", "calls_per_timing": reps},
                      "cases": res}))


# ----------------------------------------------------------------------------------- token-choice contrast
def run_contrast(args):
    """Expert choice next to the token-choice top-2 routing it is contrasted with (Section 3.1, Section 4.2), on
    identical synthetic inputs: step time (forward + backward, median of the timed regions), expert loads, dropped
    requests.  Four runs of the same layer:
      expert_choice          the paper's method, k = n*c/e slots per expert, all filled;
      token_top2             two experts per token, buffers of the same k slots, requests beyond them dropped;
      token_top2_no_drop     buffers enlarged to what the fullest expert asks for, nothing dropped; the GEMMs skip empty slots;
      fixed_shape_no_drop    what an implementation with fixed buffer shapes pays for those enlarged buffers: every
                             slot of every buffer is computed (timed as expert choice at that buffer size).
    `--expert-skew` gives some experts a popularity offset, standing in for the imbalance of a trained gate."""
    import torch
    from paper_2202_09368_b200 import binding as B
    from paper_2202_09368_b200 import inputs as IN
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    dev = torch.device("cuda")
    n, d, dff, E, c = WORKLOADS[args.workload]
    bf, chunk = torch.bfloat16, 1 << 26
    li = IN.make_layer_inputs(n, d, 8, E, bf, 0, device=dev, with_grad=False, expert_skew=args.expert_skew)
    X, Wg = li.X, li.Wg
    W1 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(d), 0, IN.TID_W1, bf, dev, chunk)
    W2 = IN.normal_tensor((E, d, dff), 1.0 / math.sqrt(dff), 0, IN.TID_W2, bf, dev, chunk)
    dY = IN.normal_tensor((n, d), 1.0, 0, IN.TID_DXOUT, bf, dev, chunk)
    X_out = torch.empty_like(X)
    grads = (torch.empty_like(X), torch.empty_like(Wg), torch.empty_like(W1), torch.empty_like(W2))

    def timed(cfg):
        ws, saved = B.alloc_workspace(cfg, dev), B.alloc_saved(cfg, dev)

        def step():
            B.ec_moe_forward(cfg, X, Wg, W1, W2, X_out, saved, ws)
            B.ec_moe_backward(cfg, X, Wg, W1, W2, dY, saved, grads, ws)
        for _ in range(max(3, args.warmup)):
            step()
        assert B.ec_read_status(ws) == B.EC_OK
        ms = []
        for _ in range(max(1, args.repeats)):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record()
            for _ in range(args.steps):
                step()
            b_.record()
            torch.cuda.synchronize()
            ms.append(a.elapsed_time(b_) / args.steps)
        assert B.ec_read_status(ws) == B.EC_OK
        v = B.saved_view(cfg, saved)
        per_token = torch.bincount((v["row_ptr"][1:] - v["row_ptr"][:-1]).long()).tolist()
        out = {"ms_per_step": round(sorted(ms)[len(ms) // 2], 4), "best_ms": round(min(ms), 4), "slots_per_expert": B.ec_capacity(cfg),
               "tokens_by_number_of_experts": per_token}
        if cfg.router:
            load, req = v["load"].view(-1).tolist(), v["requested"].view(-1).tolist()
            k = B.ec_capacity(cfg)
            out.update({"requested_min_median_max": [min(req), sorted(req)[len(req) // 2], max(req)],
                        "fullest_expert_over_buffer": round(max(req) / k, 3), "experts_over_their_buffer": sum(r > k for r in req),
                        "requests_dropped": round(1.0 - sum(load) / sum(req), 4), "filled_slots": sum(load)})
        del ws, saved
        return out, (v["requested"].max().item() if cfg.router else None)

    res = {}
    res["expert_choice"], _ = timed(B.make_config(n, d, dff, E, c, bf))
    res["token_top2"], fullest = timed(B.make_config(n, d, dff, E, c, bf, router="token"))
    c_big = (fullest + 0.5) * E / n                                # buffers of exactly what the fullest expert asked for
    res["token_top2_no_drop"], _ = timed(B.make_config(n, d, dff, E, c_big, bf, router="token"))
    res["fixed_shape_no_drop"], _ = timed(B.make_config(n, d, dff, E, c_big, bf))
    ec = res["expert_choice"]["ms_per_step"]
    print(json.dumps({"metric": "ec_vs_token_choice_step_time", "unit": "ms per forward+backward step (median region)",
                      "config": {"workload": workload_desc(args.workload), "expert_skew": args.expert_skew,
                                 "data": "synthetic; a popularity offset per expert stands in for a trained gate's imbalance",
                                 "regions": args.repeats, "steps_each": args.steps},
                      "runs": res,
                      "step_time_over_expert_choice": {k_: round(v_["ms_per_step"] / ec, 3) for k_, v_ in res.items()}}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40, help="steps per timed region")
    ap.add_argument("--repeats", type=int, default=5, help="timed regions per run; the line reports the median one")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4", choices=sorted(WORKLOADS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--graph", action="store_true", help="time the step as one captured CUDA graph")
    ap.add_argument("--cap-b", type=int, default=0, help="at most this many experts per token (Section 3.3); 0 = plain expert choice")
    ap.add_argument("--cap-iters", type=int, default=100, help="rounds of the capped solver")
    ap.add_argument("--groups", type=int, default=1, help="route the n tokens as this many independent groups")
    ap.add_argument("--fuse-gather", action="store_true", help="the expert GEMMs read the chosen rows of X in place; X_in is not written")
    ap.add_argument("--routing", action="store_true", help="routing-only stress grid instead of the layer benchmark")
    ap.add_argument("--sweep", action="store_true", help="capacity-factor sweep of the forward pass instead of the layer benchmark")
    ap.add_argument("--route-case", default="", help="with --routing: one case 'n,E' or 'n,E,d' instead of the grid")
    ap.add_argument("--gemms", action="store_true", help="the expert GEMMs alone in a loop, torch.bmm beside them (calibration)")
    ap.add_argument("--loop-seconds", type=float, default=0.0, help="with --gemms: loop every product this long and report watts, clocks and pJ per flop")
    ap.add_argument("--contrast", action="store_true", help="expert choice beside token-choice top-2 routing on identical inputs")
    ap.add_argument("--expert-skew", type=float, default=0.05, help="with --contrast: popularity offset of the experts' gate logits")
    args = ap.parse_args()
    if args.gemms:
        run_gemms(args)
    elif args.contrast:
        run_contrast(args)
    elif args.sweep:
        run_sweep(args)
    elif args.routing:
        run_routing(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()

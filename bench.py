#!/usr/bin/env python
"""Benchmark of the BigBird block-sparse attention forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One "step" is one pass of the whole hot path (layout already built; Q/K/V -> out, lse) over one batch of
the BigBird-base workload: B=8, H=12, N=4096, D=64, block 64, 3 window + 2 global + 3 random blocks, bf16.
The metric counts only the FLOPs of the attended block pairs (4*b*b*D each).  Rank 0 prints one JSON line.

With N > 1 (under torchrun) every rank runs the same workload on its own GPU (the op shards over batch and
head with no exchange, so there is no collective on the data path); the value is the total over ranks
divided by the slowest rank's time.

`--impl reference` times the fp64 CPU oracle as it stands on the host cores (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2007_14062_b200 import synth  # noqa: E402

METRIC = "block-sparse attn fwd TFLOP/s (counted FLOPs) & % bf16 TC peak at N=4096"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"bf16_tflops": 1590.0, "hbm_gbs": 6650.0}
# dram__bytes_read.sum + dram__bytes_write.sum of one attn_fwd_sm100_kernel launch on this workload, from the
# ncu capture summarised in profiles/ (None until a capture exists for the current kernel).
NCU_DRAM_BYTES_PER_LAUNCH = {"c2_base_itc_bf16": 242.1e6}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", 0)),
                "hbm_gbs": float(d["hbm_gbs"]), "source": "measured"}
    return dict(FALLBACK_PEAKS, bf16_tflops_sustained=1400.0, source="fallback")


def counted_pairs(layout) -> int:
    """Attended (query block, key block) pairs per batch element, summed over heads (the nominal count: every pair
    of the layout, App. D's cost formula O(n (g + w + r) b d))."""
    return int(layout.nnz)


def effective_pairs(layout, wl, kpm) -> int:
    """Pairs of the whole batch that survive the key-padding mask: the query block has at least one valid row and
    the key block at least one valid key.  Equal to B x nominal when nothing is padded."""
    if kpm is None:
        return wl.B * counted_pairs(layout)
    nb = wl.N // wl.b
    valid = kpm.numpy().reshape(wl.B, nb, wl.b).any(axis=2)                 # [B, nb]
    row_ptr, col_idx = layout.export()
    rows = np.repeat(np.arange(wl.H * nb), np.diff(row_ptr)) % nb          # query block of every pair
    return int((valid[:, rows] & valid[:, col_idx]).sum())


class ClockSampler:
    """Samples SM clock and clock-event reasons of the benchmarked GPU through NVML while the timed region runs."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, device_index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception as e:  # NVML missing: report that no clocks were sampled
            self.nv, self.h, self.err = None, None, repr(e)

    def _loop(self):
        nv = self.nv
        # the first sample half a millisecond in: by then the main thread has enqueued a short run's launches and
        # sits in its synchronize (without the interpreter lock), so the sampling never delays a launch
        time.sleep(0.0005)
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def max_over_ranks(values, dist, device):
    """Every rank's timings -> the slowest rank's (the job is as slow as its slowest replica).  `dist` is
    torch.distributed or None for a single process."""
    if dist is None:
        return [float(v) for v in values]
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t]


def whole_job_value(per_replica_units, world, slowest_ms):
    """Aggregate throughput of `world` replicas that each process `per_replica_units` per step."""
    return world * per_replica_units / (slowest_ms * 1e-3)


def workload_config(wl, pairs_per_batch):
    """The keys both arms report for the workload (same names, same values)."""
    return {"workload": wl.name, "B": wl.B, "H": wl.H, "N": wl.N, "D": wl.D, "block": wl.b, "window_blocks": wl.w,
            "global_blocks": wl.g, "random_blocks": wl.r, "mode": "ETC" if wl.mode else "ITC",
            "attended_block_pairs_per_step": wl.B * pairs_per_batch,
            "counted_gflop_per_step": wl.B * pairs_per_batch * 4.0 * wl.b * wl.b * wl.D / 1e9}


def oracle_slices(wl, q, k, v, kpm, slices):
    from oracle import bigbird_oracle as O
    gr = O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    t0 = time.perf_counter()
    res = O.attention(q, k, v, gr, kpm, wl.scale, slices=slices)
    return time.perf_counter() - t0, res


def cpu_baseline(wl, pairs_per_batch, gpu_out=None, gpu_lse=None, budget_s=12.0):
    """Times the oracle, as it stands, on a bounded sample of (batch, head) slices of the workload, and compares
    the library's output for those slices (batch element 0 of the first input set) with it."""
    q, k, v = synth.make_qkv(wl, batch_limit=1)
    qn, kn, vn = (t.float().numpy() for t in (q, k, v))
    kpm = synth.key_padding_mask(wl)
    kp = None if kpm is None else kpm.numpy()
    flops_per_slice = pairs_per_batch / wl.H * 4.0 * wl.b * wl.b * wl.D
    t1, _ = oracle_slices(wl, qn, kn, vn, kp, [(0, 0)])
    n = int(max(1, min(wl.H - 1, budget_s / max(t1, 1e-3))))
    slices = [(0, 1 + i) for i in range(n)] if wl.H > 1 else [(0, 0)]
    t, res = oracle_slices(wl, qn, kn, vn, kp, slices)
    cores = len(os.sched_getaffinity(0))
    out = {"value": flops_per_slice * len(slices) / t / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
           "sample": f"{len(slices)} of {wl.B * wl.H} (batch, head) slices at full N={wl.N}, fp64 masked dense attention; "
                     f"{t / len(slices):.3f} s per slice",
           "seconds_per_slice": t / len(slices)}
    if gpu_out is not None:
        valid = np.ones(wl.N, dtype=bool) if kp is None else kp[0] != 0
        eo = el = 0.0
        for (bi, h), (wo, wlse) in res.items():
            eo = max(eo, float(np.abs(gpu_out[h][valid] - wo[valid]).max()))
            el = max(el, float(np.abs(gpu_lse[h][valid] - wlse[valid]).max()))
        out["max_abs_err_out_vs_oracle"] = eo
        out["max_abs_err_lse_vs_oracle"] = el
    return out


def run_reference(args, wl):
    """The oracle as the reference arm: each step is one (batch, head) slice at full sequence length."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import bigbird_oracle as O
    # attended block pairs counted from the oracle's own mask: nothing of the CUDA library is on this arm
    row_ptr, _ = O.layout_from_mask(O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode))
    flops_per_slice = int(row_ptr[-1]) / wl.H * 4.0 * wl.b * wl.b * wl.D
    q, k, v = synth.make_qkv(wl, batch_limit=1)
    qn, kn, vn = (t.float().numpy() for t in (q, k, v))
    kpm = synth.key_padding_mask(wl)
    kp = None if kpm is None else kpm.numpy()
    for i in range(args.warmup):
        oracle_slices(wl, qn, kn, vn, kp, [(0, i % wl.H)])
    t = 0.0
    for i in range(args.steps):
        t += oracle_slices(wl, qn, kn, vn, kp, [(0, i % wl.H)])[0]
    value = flops_per_slice * args.steps / t / 1e12
    cores = len(os.sched_getaffinity(0))
    sample = f"each step = 1 of {wl.B * wl.H} (batch, head) slices at full N={wl.N} (fp64 masked dense attention on the host)"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": dict(workload_config(wl, int(row_ptr[-1])), sample=sample),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_backward(args, wl):
    """`--direction bwd`: the gradient kernels (CUDA cores, fp32 arithmetic) on the same workload, one GPU.  Their
    FLOPs are counted like the forward pass's: five b x b x D products per attended block pair (the scores again,
    dP, dV, dQ, dK) against the forward pass's two."""
    import paper_2007_14062_b200 as bb
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    steps = 20 if args.steps is None else args.steps
    warmup = max(3, 3 if args.warmup is None else args.warmup)
    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    pairs = counted_pairs(L)
    flops_per_step = wl.B * pairs * 10.0 * wl.b * wl.b * wl.D
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    gen = torch.Generator().manual_seed(wl.seed + 100)
    dout = torch.randn(q.shape, generator=gen, dtype=torch.float32).to(q.dtype)
    qd, kd, vd, dod = (t.to(dev) for t in (q, k, v, dout))
    md = None if kpm is None else kpm.to(dev)
    out, lse = torch.empty_like(qd), torch.empty(q.shape[:3], device=dev, dtype=torch.float32)
    bb.bigbird_attn_fwd(qd, kd, vd, L, md, out, lse, wl.scale)
    dq, dk, dv = (torch.empty_like(qd) for _ in range(3))
    stream = torch.cuda.current_stream(dev)

    def step():
        bb.bigbird_attn_bwd(qd, kd, vd, out, lse, dod, L, md, dq, dk, dv, wl.scale, stream.cuda_stream)

    for _ in range(warmup):
        step()
    launches = bb.bigbird_last_launch_count()
    sampler = ClockSampler(0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    sampler.start()
    ev0.record(stream)
    for _ in range(steps):
        step()
    ev1.record(stream)
    torch.cuda.synchronize()
    sampler.stop()
    ms_per_step = ev0.elapsed_time(ev1) / steps
    tflops = flops_per_step / (ms_per_step * 1e-3) / 1e12
    clocks = sampler.summary()
    # fp32 FMA peak of the CUDA cores from unit counts and the clock: SMs x 128 lanes x 2 FLOP x max SM clock
    sms = torch.cuda.get_device_properties(dev).multi_processor_count
    alu_peak = sms * 128 * 2 * (clocks["sm_max_mhz"] or 1965) * 1e6 / 1e12
    elt = q.element_size()
    min_bytes = wl.B * wl.H * wl.N * (8 * wl.D * elt + 4)          # q, k, v, out, dout read, dq, dk, dv written, lse read
    line = {"metric": "block-sparse attn bwd TFLOP/s (counted FLOPs)", "value": tflops, "unit": UNIT, "n_gpus": 1, "steps": steps,
            "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic", "direction": "bwd",
            "config": dict(workload_config(wl, pairs), counted_gflop_per_step_bwd=flops_per_step / 1e9,
                           l2=f"one set of eight tensors ({8 * q.numel() * elt / 1e6:.0f} MB)"),
            "gpu_launches": launches * steps, "clocks": clocks,
            "roofline": {"bound": "alu", "achieved": tflops, "peak": alu_peak, "unit": "TFLOP/s", "frac": tflops / alu_peak,
                         "traffic": None, "peak_source": "fp32 FMA lanes x clock (derived)", "kernel": "attn_bwd_dq_kernel + attn_bwd_dkv_kernel",
                         "min_hbm_bytes_per_launch": min_bytes, "achieved_hbm_gbs_on_min_bytes": min_bytes / (ms_per_step * 1e-3) / 1e9}}
    if not args.no_cpu_baseline:
        from oracle import bigbird_oracle as O
        gr = O.Graph(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
        t0 = time.perf_counter()
        want = O.attention_bwd(q[:1].float().numpy(), k[:1].float().numpy(), v[:1].float().numpy(), dout[:1].float().numpy(), gr,
                               None if kpm is None else kpm[:1].numpy(), wl.scale, slices=[(0, 0)])
        t = time.perf_counter() - t0
        got = [x[0, 0].float().cpu().numpy() for x in (dq, dk, dv)]
        err = max(float(np.abs(g - w_).max()) for g, w_ in zip(got, want[(0, 0)]))
        line["cpu_baseline"] = {"value": flops_per_step / (wl.B * wl.H) / t / 1e12, "unit": UNIT, "cores": len(os.sched_getaffinity(0)),
                                "kind": "oracle", "sample": f"1 of {wl.B * wl.H} (batch, head) slices, fp64 gradients; {t:.2f} s",
                                "max_abs_err_grads_vs_oracle": err}
    print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None, help="timed steps (default 200; 12 for --impl reference)")
    ap.add_argument("--warmup", type=int, default=None, help="untimed steps before them (default 50; 3 for --impl reference)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2_base_itc_bf16", choices=synth.ORDER)
    ap.add_argument("--e2e-steps", type=int, default=20)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--direction", default="fwd", choices=["fwd", "bwd"], help="bwd: time the gradient kernels instead (one GPU)")
    args = ap.parse_args()
    wl = synth.WORKLOADS[args.workload]

    if args.impl == "reference":
        args.steps = 12 if args.steps is None else args.steps
        args.warmup = 3 if args.warmup is None else args.warmup
        run_reference(args, wl)
        return
    if args.direction == "bwd":
        if int(os.environ.get("RANK", "0")) == 0:
            run_backward(args, wl)
        return
    args.steps = 200 if args.steps is None else args.steps
    # at least 20 warm-up steps whatever was asked for (3 ms of this kernel: the clock ramp after idle, see below);
    # the JSON line reports the number actually run
    args.warmup = max(20, 50 if args.warmup is None else args.warmup)

    import paper_2007_14062_b200 as bb

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    L = bb.bigbird_build_layout(wl.N, wl.b, wl.w, wl.g, wl.r, wl.seed, wl.H, wl.mode)
    pairs = counted_pairs(L)
    flops_per_step = wl.B * pairs * 4.0 * wl.b * wl.b * wl.D
    tokens_per_step = wl.B * wl.N

    # Rotating input sets so that no step finds its inputs in L2 (4 sets x 201 MB for the base workload; L2 is 126 MB).
    q, k, v = synth.make_qkv(wl)
    kpm = synth.key_padding_mask(wl)
    eff_pairs = effective_pairs(L, wl, kpm)
    eff_flops_per_step = eff_pairs * 4.0 * wl.b * wl.b * wl.D
    n_sets = 4
    sets = []
    for i in range(n_sets):
        qd, kd, vd = (t.to(dev) for t in (q, k, v))
        if i:
            qd, kd, vd = qd.roll(i, 0), kd.roll(i, 0), vd.roll(i, 0)          # same values, other batch order
        md = None if kpm is None else kpm.roll(i, 0).to(dev).contiguous()
        sets.append((qd.contiguous(), kd.contiguous(), vd.contiguous(), md, torch.empty_like(qd),
                     torch.empty(q.shape[:3], device=dev, dtype=torch.float32)))
    stream = torch.cuda.current_stream(dev)

    def step(i):
        qd, kd, vd, md, od, ld = sets[i % n_sets]
        bb.bigbird_attn_fwd(qd, kd, vd, L, md, od, ld, wl.scale, stream.cuda_stream)

    # Everything that takes host time (NVML start-up, event creation) comes before the warm-up, and nothing but the
    # barrier sits between the warm-up and the timed region: a GPU left idle for a few milliseconds drops its clocks
    # and needs about ten launches (1.5 ms) to come back, which a short timed region would otherwise be charged with.
    sampler = ClockSampler(local_rank)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for i in range(args.warmup):
        step(i)
    launches_per_step = bb.bigbird_last_launch_count()
    barrier()
    sampler.start()
    ev0.record(stream)
    for i in range(args.steps):
        step(i)
    ev1.record(stream)
    barrier()
    sampler.stop()
    ms = ev0.elapsed_time(ev1)
    st, detail = bb.bigbird_last_status(stream.cuda_stream)
    if st != 0:
        raise SystemExit(f"kernel reported status {st} (wait {detail})")

    # ---- end to end: pinned host buffers in, results back to the host, every step ----
    hq, hk, hv = (t.pin_memory() for t in (q, k, v))
    hm = None if kpm is None else kpm.pin_memory()
    ho = torch.empty_like(q).pin_memory()
    hl = torch.empty(q.shape[:3], dtype=torch.float32).pin_memory()
    dq, dk, dv, dm, do, dl_ = sets[0]

    # The batch goes through in slices on three streams (copies in, compute, copies out), so that the PCIe
    # transfers of one slice overlap the other direction's transfers and the kernel of its neighbours.
    n_slices = min(wl.B, 4)
    bounds = [(wl.B * i // n_slices, wl.B * (i + 1) // n_slices) for i in range(n_slices)]
    s_in, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    ev_in = [torch.cuda.Event() for _ in bounds]
    ev_cmp = [torch.cuda.Event() for _ in bounds]
    ev_out = [torch.cuda.Event() for _ in bounds]

    def e2e_step():
        for c, (b0, b1) in enumerate(bounds):
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_cmp[c])            # the previous step's kernel has read this slice
                dq[b0:b1].copy_(hq[b0:b1], non_blocking=True)
                dk[b0:b1].copy_(hk[b0:b1], non_blocking=True)
                dv[b0:b1].copy_(hv[b0:b1], non_blocking=True)
                if hm is not None:
                    dm[b0:b1].copy_(hm[b0:b1], non_blocking=True)
                ev_in[c].record(s_in)
            stream.wait_event(ev_in[c])
            stream.wait_event(ev_out[c])              # the previous step's results of this slice have left
            bb.bigbird_attn_fwd(dq[b0:b1], dk[b0:b1], dv[b0:b1], L, None if dm is None else dm[b0:b1], do[b0:b1], dl_[b0:b1],
                                wl.scale, stream.cuda_stream)
            ev_cmp[c].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[c])
                ho[b0:b1].copy_(do[b0:b1], non_blocking=True)
                hl[b0:b1].copy_(dl_[b0:b1], non_blocking=True)
                ev_out[c].record(s_out)

    def e2e_join():
        for c in range(len(bounds)):
            stream.wait_event(ev_out[c])

    for _ in range(3):
        e2e_step()
    e2e_join()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    s_in.wait_event(e0)
    for _ in range(args.e2e_steps):
        e2e_step()
    e2e_join()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hv)) + (0 if hm is None else hm.numel())
    d2h = ho.numel() * ho.element_size() + hl.numel() * 4

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], dist, dev)

    if rank == 0:
        peaks = measured_peaks()
        ms_per_step = ms / args.steps
        tflops = whole_job_value(flops_per_step, world, ms_per_step) / 1e12
        per_gpu = tflops / world
        e2e_tflops = world * flops_per_step / (e2e_ms / args.e2e_steps * 1e-3) / 1e12
        traffic = NCU_DRAM_BYTES_PER_LAUNCH.get(wl.name)
        min_bytes = wl.B * wl.H * wl.N * (4 * wl.D * (2 if wl.dtype == 'bf16' else 4) + 4)
        line = {
            "metric": METRIC, "value": tflops, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
            "config": dict(workload_config(wl, pairs),
                           effective_block_pairs_per_step=eff_pairs, effective_gflop_per_step=eff_flops_per_step / 1e9,
                           l2=f"rotating {n_sets} input/output sets ({n_sets * 4 * q.numel() * q.element_size() / 1e6:.0f} MB) larger than L2",
                           parallelism=f"replicas x{world}" if world > 1 else "single GPU"),
            "tokens_per_s": world * tokens_per_step / (ms_per_step * 1e-3),
            # the same time against the pairs that survive the key-padding mask (equal to `value` without padding)
            "effective_tflops": tflops * eff_flops_per_step / flops_per_step,
            "pct_of_measured_bf16_peak_effective": 100.0 * per_gpu * eff_flops_per_step / flops_per_step / peaks["bf16_tflops"],
            "pct_of_measured_bf16_peak": 100.0 * per_gpu / peaks["bf16_tflops"],
            "pct_of_nominal_bf16_peak": 100.0 * per_gpu / NOMINAL_BF16_TFLOPS,
            "e2e": {"value": e2e_tflops, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "steps": args.e2e_steps, "ms_per_step": e2e_ms / args.e2e_steps,
                    "how": f"pinned host buffers, batch in {n_slices} slices on three streams (copies in / kernel / copies out)"},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": sampler.summary(),
            "roofline": {"bound": "tensor", "achieved": per_gpu, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": per_gpu / peaks["bf16_tflops"], "traffic": traffic,
                         "peak_source": f"{peaks['source']} bf16 burst", "kernel": "attn_fwd_sm100_kernel" if wl.dtype == "bf16" else "attn_fwd_simt_kernel",
                         "kernel_us": 1e3 * ms_per_step, "algorithmic_flops_per_launch": flops_per_step,
                         "min_hbm_bytes_per_launch": min_bytes,
                         "achieved_hbm_gbs_on_min_bytes": min_bytes / (ms_per_step * 1e-3) / 1e9,
                         "frac_of_sustained_peak": per_gpu / peaks["bf16_tflops_sustained"] if peaks["bf16_tflops_sustained"] else None},
        }
        if world == 1 and not args.no_cpu_baseline:
            # batch element 0 of the first input set holds the workload's own (unrolled) tensors
            step(0)
            torch.cuda.synchronize()
            line["cpu_baseline"] = cpu_baseline(wl, pairs, sets[0][4][0].float().cpu().numpy(), sets[0][5][0].cpu().numpy())
        print(json.dumps(line))
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

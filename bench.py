#!/usr/bin/env python
"""Benchmark of the ReLU linear-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload 480p|720p]
                    [--shard replicas|tokens]

One step = one pass of the bidirectional hot path (state reduction over K,V + apply over Q, writing
bf16 O) over one batch of seeded synthetic input shaped like a 480p 5-second latent (20 heads x 112,
32760 tokens).  The metric is linear-attention tokens*heads per second.  Rank 0 prints ONE JSON line.

`--impl reference` times the fp64 CPU oracle (the only reference that exists for this method) on the
host cores, on a bounded sample of the same workload.

With N > 1 (torchrun) every rank runs the same per-GPU workload on its own GPU (independent batch
shards, no data-path collective): weak scaling, value = all ranks' tokens*heads / max-over-ranks time.
`--shard tokens` instead splits the ONE sequence by tokens over the ranks: each rank reduces its shard's
state, one all-reduce (sum) of the ~1 MB state follows, each rank applies its own queries (strong scaling).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

# dram__bytes_read.sum + dram__bytes_write.sum per forward launch, from the ncu capture summarised under
# profiles/ (None once the kernel has changed since the counters were taken)
NCU_TRAFFIC_BYTES = {"480p_5s_bidir": 556.3e6}
# the same for side workloads whose dominant launch was captured (keys of roofline.per_workload)
NCU_TRAFFIC_SIDE = {"720p_minute_stream_step": 362.9e6, "480p_5s_bidir_rope": 574.0e6}

METRIC = "linear_attn_tokens_heads_per_s"
UNIT = "tokens*heads/s"


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="480p", choices=["480p", "720p"])
    ap.add_argument("--shard", default="replicas", choices=["replicas", "tokens"],
                    help="N > 1: independent replicas (weak scaling) or one sequence split by tokens (strong scaling)")
    ap.add_argument("--no-extras", action="store_true", help="skip the block-step / 720p side measurements")
    ap.add_argument("--kernels-only", action="store_true",
                    help="time the device kernels only (no host-buffer leg, no CPU oracle, no side measurements): "
                         "the short command used under a profiler")
    return ap.parse_args()


def workload_of(name):
    import synth

    return synth.P480 if name == "480p" else synth.P720


def peaks():
    """Measured HBM copy bandwidth of this machine's B200s, else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML (read-only) while the timed region runs."""

    def __init__(self, index: int):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksEventReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                try:
                    bits = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    bits = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in names.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def cpu_oracle_throughput(w, budget_s, q, k, v):
    """The oracle as it stands on a bounded sample: every head, the first n_s tokens of the workload."""
    import oracle

    orc = oracle.default()
    cores = min(os.cpu_count() or 1, w.B * w.H)  # the oracle parallelises over (batch, head) units only
    n_s = min(w.N, 2048)
    t0 = time.perf_counter()
    orc.forward(q[:, :n_s], k[:, :n_s], v[:, :n_s], w.eps)
    t_probe = time.perf_counter() - t0
    n_s = int(max(256, min(w.N, n_s * budget_s / max(t_probe, 1e-4))))
    t0 = time.perf_counter()
    orc.forward(q[:, :n_s], k[:, :n_s], v[:, :n_s], w.eps)
    dt = time.perf_counter() - t0
    # one thread: the oracle parallelises over (batch, head) units only, so one unit runs on one core
    n_1 = max(256, n_s // 4)
    q1, k1, v1 = (np.ascontiguousarray(x[:1, :n_1, :1]) for x in (q, k, v))
    t0 = time.perf_counter()
    orc.forward(q1, k1, v1, w.eps)
    dt1 = time.perf_counter() - t0
    return {"value": w.B * n_s * w.H / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"fp64 oracle forward over all {w.B * w.H} (batch,head) units, first {n_s} of {w.N} tokens, "
                      f"{dt:.2f} s wall",
            "one_thread": {"value": n_1 / dt1, "unit": UNIT, "sample": f"one (batch, head) unit, first {n_1} tokens, "
                                                                        f"{dt1:.2f} s wall"}}, n_s


def run_reference(args):
    """--impl reference: the CPU oracle, rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import synth
    import oracle

    w = workload_of(args.workload)
    orc = oracle.default()
    q, k, v = synth.qkv(w)
    # size the per-step sample so that steps+warmup stay within about two minutes
    n_s = min(w.N, 1024)
    t0 = time.perf_counter()
    orc.forward(q[:, :n_s], k[:, :n_s], v[:, :n_s], w.eps)
    per_tok = (time.perf_counter() - t0) / n_s
    n_s = int(max(128, min(w.N, 120.0 / max(1, args.steps + args.warmup) / per_tok)))
    qs, ks, vs = q[:, :n_s], k[:, :n_s], v[:, :n_s]
    for _ in range(args.warmup):
        orc.forward(qs, ks, vs, w.eps)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        orc.forward(qs, ks, vs, w.eps)
    dt = time.perf_counter() - t0
    value = args.steps * w.B * n_s * w.H / dt
    cores = min(os.cpu_count() or 1, w.B * w.H)
    sample = f"fp64 oracle forward, all {w.B * w.H} units, first {n_s} of {w.N} tokens per step"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "d": w.d, "N": w.N, "sample_tokens_per_step": n_s},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def max_over_ranks(torch, dist, ms: float, device) -> float:
    """A multi-rank time is the slowest rank's: all-reduce MAX (NCCL on GPUs, gloo in the CPU tests)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(world: int, units_per_rank: int, ms_per_step: float) -> float:
    """Weak scaling: every rank processes `units_per_rank` tokens*heads per step on its own shard."""
    return world * units_per_rank / (ms_per_step * 1e-3)


NOMINAL_HBM_GBS = 8000.0   # the "~8 TB/s" the B200 data sheet names; the measured copy peak is the roofline's denominator


def frac_entry(us: float, nbytes: float, peak: float) -> dict:
    """One compact line of the per-workload roofline: time, algorithmic GB/s, fraction of the measured copy peak
    and of the nominal 8 TB/s."""
    gbs = nbytes / (us * 1e-6) / 1e9
    return {"us": round(us, 2), "gbs": round(gbs, 1), "frac": round(gbs / peak, 4), "frac_8tbs": round(gbs / NOMINAL_HBM_GBS, 4)}


def time_loop(torch, fn, steps, sync_ranks=None):
    """CUDA-event time of `steps` calls of fn(i) on the current stream, in ms."""
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if sync_ranks:
        sync_ranks()
    torch.cuda.synchronize()
    start.record()
    for i in range(steps):
        fn(i)
    stop.record()
    torch.cuda.synchronize()
    if sync_ranks:
        sync_ranks()
    return start.elapsed_time(stop)


def main():
    args = parse()
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import paper_2509_24695_b200 as la
    import synth

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod

        dist = dist_mod
        dist.init_process_group("nccl")
    sync_ranks = (lambda: dist.barrier()) if dist else None

    la.load_library()
    w = workload_of(args.workload)
    K, W = args.steps, max(args.warmup, 3)
    dev = torch.device("cuda", local_rank)
    shard_tokens = args.shard == "tokens"

    # seeded synthetic inputs (same bits the oracle sees); two rotating input sets so no step finds
    # its inputs in L2 (one set is 4 x 147 MB = 587 MB at 480p, already > 126 MB of L2)
    q_h, k_h, v_h = synth.qkv(w)
    if shard_tokens:
        # ONE sequence split by tokens: this rank holds rows [lo, hi) of Q, K, V and produces those rows of O
        from paper_2509_24695_b200 import sharded

        lo, hi = sharded.shard_bounds(w.N, world, rank, multiple=128)
        q_h, k_h, v_h = (np.ascontiguousarray(x[:, lo:hi]) for x in (q_h, k_h, v_h))

    def dev_of(bits):
        return torch.from_numpy(bits.view("int16")).to(dev).view(torch.bfloat16)

    sets = []
    for r in range(2):
        qd, kd, vd = dev_of(q_h), dev_of(k_h), dev_of(v_h)
        if r:  # second set: same distribution, other values (token order reversed)
            qd, kd, vd = qd.flip(1).contiguous(), kd.flip(1).contiguous(), vd.flip(1).contiguous()
        sets.append((qd, kd, vd, torch.empty_like(qd)))
    ws = la.new_workspace(sets[0][0])
    units = w.B * w.N * w.H  # tokens*heads per step (of the whole sequence)
    local_units = w.B * q_h.shape[1] * w.H

    if shard_tokens:
        shard_state = torch.empty((w.B, w.H, w.d + 1, w.d), dtype=torch.float32, device=dev)

        def step(i):
            qd, kd, vd, od = sets[i & 1]
            # state of this rank's tokens -> one all-reduce (sum) of ~1 MB into this rank's buffer -> apply to its queries
            sharded.linattn_forward_token_sharded(
                qd, kd, vd, w.eps, state_fn=lambda k_, v_: la.linattn_state(k_, v_, out=shard_state, workspace=ws),
                apply_fn=lambda q_, st: la.linattn_apply(q_, st, w.eps, out=od, workspace=ws))
    else:
        def step(i):
            qd, kd, vd, od = sets[i & 1]
            la.linattn_forward(qd, kd, vd, w.eps, out=od, workspace=ws)

    for i in range(W):
        step(i)
    sampler = ClockSampler(local_rank)
    sampler.start()
    l0 = la.kernel_launches()
    ms = time_loop(torch, step, K, sync_ranks)
    launches = la.kernel_launches() - l0
    # keep the device busy until the sampler has seen the clocks under this load
    t_end = time.time() + 0.25
    while len(sampler.samples) < 8 and time.time() < t_end:
        step(0)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    ms = max_over_ranks(torch, dist, ms, dev)
    ms_per_step = ms / K
    # replicas: every rank runs the whole workload on its own data; tokens: the ranks share ONE sequence
    value = units / (ms_per_step * 1e-3) if shard_tokens else whole_job_value(world, units, ms_per_step)

    # The library launches ONE kernel per call (state pass + split-N reduce + apply pass fused), so the
    # dominant kernel is the forward launch itself: algorithmic bytes = 8d per token*head (read q, k, v,
    # write o), duration = the CUDA-event time per step measured above.  The two passes are also timed
    # alone (same kernel, one pass switched off), for reference.
    state_buf = la.linattn_state(sets[0][1], sets[0][2], workspace=ws)
    ms_state = time_loop(torch, lambda i: la.linattn_state(sets[i & 1][1], sets[i & 1][2], out=state_buf, workspace=ws), K) / K
    ms_apply = time_loop(torch, lambda i: la.linattn_apply(sets[i & 1][0], state_buf, w.eps, out=sets[i & 1][3], workspace=ws), K) / K
    peak, peak_kind = peaks()
    bytes_tok_head = 2 * w.d  # one bf16 row of d features
    state_bytes = la.state_bytes(w.B, w.H, w.d)
    kern = {
        "state": {"ms": ms_state, "bytes": local_units * 2 * bytes_tok_head + state_bytes},      # read K, V; write state
        "apply": {"ms": ms_apply, "bytes": local_units * 2 * bytes_tok_head + state_bytes},      # read Q, state; write O
        "forward": {"ms": ms_per_step, "bytes": local_units * 4 * bytes_tok_head},               # 8d bytes per token*head
    }
    for kv in kern.values():
        kv["gbs"] = kv["bytes"] / (kv["ms"] * 1e-3) / 1e9
    roofline = {"bound": "hbm",
                "kernel": f"umma_fused_kernel<{w.d}> (" + ("linattn_state + all-reduce + linattn_apply per step, this rank's shard)"
                                                         if shard_tokens else "linattn_forward, one launch per step)"),
                "achieved": kern["forward"]["gbs"], "peak": peak, "unit": "GB/s",
                "frac": kern["forward"]["gbs"] / peak, "peak_kind": f"of {peak_kind}",
                "bytes_per_launch": kern["forward"]["bytes"],
                "frac_8tbs": kern["forward"]["gbs"] / NOMINAL_HBM_GBS,
                "traffic": None if shard_tokens else NCU_TRAFFIC_BYTES.get(w.name),
                "passes_alone": {k_: {"ms": round(v_["ms"], 5), "gbs": round(v_["gbs"], 1), "frac": round(v_["gbs"] / peak, 4)}
                                 for k_, v_ in kern.items() if k_ != "forward"}}

    e2e = None
    if not args.kernels_only:
        # end to end through the host-buffer entry point: pinned host Q,K,V in, O out, copies inside the timed region
        pin = lambda bits: torch.from_numpy(bits.view("int16")).view(torch.bfloat16).pin_memory()
        qp, kp, vp = pin(q_h), pin(k_h), pin(v_h)
        op = torch.empty_like(qp).pin_memory()
        k_e2e = max(3, min(K, 20))
        if shard_tokens:
            # this rank's shard up from pinned memory, the sharded step, this rank's rows of O down
            def hf(qp_, kp_, vp_, op_, eps_):
                qd, kd, vd, od = sets[0]
                qd.copy_(qp_, non_blocking=True); kd.copy_(kp_, non_blocking=True); vd.copy_(vp_, non_blocking=True)
                step(0)
                op_.copy_(od, non_blocking=True)
            h2d, d2h = 3 * qp.numel() * 2, qp.numel() * 2
        else:
            hf = la.HostForward(w.B, w.N, w.H, w.d, torch.bfloat16, dev)
            h2d, d2h = hf.h2d_bytes, hf.d2h_bytes
        for _ in range(2):
            hf(qp, kp, vp, op, w.eps)
        ms_e2e = time_loop(torch, lambda i: hf(qp, kp, vp, op, w.eps), k_e2e, sync_ranks)
        ms_e2e = max_over_ranks(torch, dist, ms_e2e, dev)
        e2e_value = units / (ms_e2e / k_e2e * 1e-3) if shard_tokens else whole_job_value(world, units, ms_e2e / k_e2e)
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": k_e2e, "ms_per_step": ms_e2e / k_e2e}
        assert float(op.float().abs().sum()) > 0.0

    out = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if shard_tokens else "weak",
        "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "H": w.H, "d": w.d, "N": w.N, "eps": w.eps,
                   "l2": "two rotating input sets of 587 MB each (> 126 MB L2)" if args.workload == "480p"
                   else "two rotating input sets, each far larger than L2",
                   "parallelism": (f"one sequence split by tokens over {world} ranks, one all-reduce of the state per step"
                                   if shard_tokens else f"replicas x{world}" if world > 1 else "single GPU")},
        "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
    }

    if rank == 0 and world == 1 and not args.kernels_only:
        cb, _ = cpu_oracle_throughput(w, 15.0, q_h, k_h, v_h)
        out["cpu_baseline"] = cb
        if not args.no_extras:
            ex = extras(torch, la, synth, dev, peak)
            out["other_workloads"] = ex
            # every hot-path workload in one compact place, each against the measured
            # copy peak ("frac") and against the nominal 8 TB/s ("frac_8tbs")
            pw = {w.name + "_forward": frac_entry(ms_per_step * 1e3, kern["forward"]["bytes"], peak),
                  w.name + "_state_alone": frac_entry(ms_state * 1e3, kern["state"]["bytes"], peak),
                  w.name + "_apply_alone": frac_entry(ms_apply * 1e3, kern["apply"]["bytes"], peak)}
            for name, e in ex.items():
                if "step_latency_us" in e and "tokens_per_block" in e:
                    by = e["algorithmic_gbs"] * e["step_latency_us"] * 1e3
                    pw[name + "_step"] = frac_entry(e["step_latency_us"], by, peak)
                    pw[name + "_step_graph"] = frac_entry(e["step_latency_us_graph_replay"], by, peak)
                    if "step_latency_us_rope" in e:
                        pw[name + "_step_rope"] = frac_entry(e["step_latency_us_rope"], by, peak)
                elif "ms" in e and "algorithmic_gbs" in e:
                    pw[name] = frac_entry(e["ms"] * 1e3, e["algorithmic_gbs"] * e["ms"] * 1e6, peak)
                elif "step_latency_us" in e and "algorithmic_gbs" in e:
                    pw[name] = frac_entry(e["step_latency_us"], e["algorithmic_gbs"] * e["step_latency_us"] * 1e3, peak)
            for name, traffic in NCU_TRAFFIC_SIDE.items():
                if name in pw:
                    pw[name]["traffic"] = traffic
            roofline["per_workload"] = pw
    if rank == 0:
        print(json.dumps(out))
    if dist:
        dist.destroy_process_group()


def extras(torch, la, synth, dev, peak):
    """Side measurements: block-step latency of the autoregressive and streaming configs (cache bytes stay
    constant as blocks accumulate) and the 720p bidirectional layer."""
    res = {}
    for w, n_steps in ((synth.AR480, 21), (synth.STREAM720, 80)):
        # a few distinct blocks, cycled: the cost of a step does not depend on the values
        blocks = []
        for b in range(3):
            qb, kb, vb = synth.qkv_block(w, b)
            blocks.append(tuple(torch.from_numpy(x.view("int16")).to(dev).view(torch.bfloat16) for x in (qb, kb, vb)))
        ob = torch.empty_like(blocks[0][0])
        cache = la.BlockLinCache(w.B, w.H, w.d, torch.bfloat16, dev, max_T_b=w.T_b, eps=w.eps)
        for i in range(3):
            cache.step(*blocks[i % 3], out=ob)
        cache.reset()
        # timed through the C entry point with prebuilt pointers: the host side of a step stays well below the
        # device time, so the events measure the device
        import ctypes
        lib = la.load_library()
        ptrs = [tuple(ctypes.c_void_p(t.data_ptr()) for t in blk) for blk in blocks]
        op, stream = ctypes.c_void_p(ob.data_ptr()), ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
        torch.cuda.synchronize()
        evs[0].record()
        for i in range(n_steps):
            qp, kp, vp_ = ptrs[i % 3]
            if lib.blocklin_step(cache._handle, w.T_b, qp, kp, vp_, op, stream) != 0:
                raise RuntimeError("blocklin_step failed")
            evs[i + 1].record()
        torch.cuda.synchronize()
        lat = [evs[i].elapsed_time(evs[i + 1]) * 1e3 for i in range(n_steps)]
        step_bytes = w.B * w.T_b * w.H * 8 * w.d + 2 * cache.info()["state_bytes"]
        med = sorted(lat)[len(lat) // 2]

        # the same steps without an event between them (an event record between two launches costs the device
        # 2-3 us): two events around the whole run, first launched one by one, then replayed from a CUDA graph
        def all_steps(handle):
            for i in range(n_steps):
                qp, kp, vp_ = ptrs[i % 3]
                if lib.blocklin_step(cache._handle, w.T_b, qp, kp, vp_, op, handle) != 0:
                    raise RuntimeError("blocklin_step failed")

        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            handle = ctypes.c_void_p(side.cuda_stream)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            all_steps(handle)
            torch.cuda.synchronize()
            e0.record(side); all_steps(handle); e1.record(side)
            torch.cuda.synchronize()
            us_launched = e0.elapsed_time(e1) * 1e3 / n_steps
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                all_steps(ctypes.c_void_p(torch.cuda.current_stream().cuda_stream))
            graph.replay()
            torch.cuda.synchronize()
            e0.record(side); graph.replay(); e1.record(side)
            torch.cuda.synchronize()
            us_graph = e0.elapsed_time(e1) * 1e3 / n_steps
        torch.cuda.current_stream().wait_stream(side)
        if la.workspace_status(cache.workspace) != 0:
            raise RuntimeError("a block step reported an error status")
        res[w.name] = {"step_latency_us": us_launched, "step_latency_us_graph_replay": us_graph,
                       "step_latency_us_median": med, "step_latency_us_first": lat[0], "step_latency_us_last": lat[-1],
                       "note": "step_latency_us: %d steps launched back to back, two events around the run; "
                               "graph_replay: the same steps replayed from one CUDA graph; median/first/last: "
                               "with an event recorded after every step" % n_steps,
                       "steps": n_steps, "tokens_per_block": w.T_b, "B": w.B,
                       "tokens_heads_per_s": w.B * w.T_b * w.H / (us_launched * 1e-6),
                       "algorithmic_gbs": step_bytes / (us_launched * 1e-6) / 1e9,
                       "frac_of_peak": step_bytes / (us_launched * 1e-6) / 1e9 / peak,
                       "frac_of_peak_graph_replay": step_bytes / (us_graph * 1e-6) / 1e9 / peak,
                       "cache_bytes_at_first_and_last_step": [cache.info()["state_bytes"]] * 2,
                       "l2": "block set of %.0f MB cycled over 3 copies" % (step_bytes / 1e6)}
        del graph
        if w.name == synth.STREAM720.name:
            # the same steps with the rotary factors of Eq. 2 (blocklin_step_rope); the block's rows of a 3D table
            cos, sin = synth.rope_table(3, 45, 80, w.d)
            table = la.rope_pack(torch.from_numpy(cos).to(dev), torch.from_numpy(sin).to(dev))
            for i in range(3):
                cache.step_rope(*blocks[i % 3], table, out=ob)
            tp = ctypes.c_void_p(table.data_ptr())

            def rope_steps(i):
                qp, kp, vp_ = ptrs[i % 3]
                if lib.blocklin_step_rope(cache._handle, w.T_b, qp, kp, vp_, op, tp, stream) != 0:
                    raise RuntimeError("blocklin_step_rope failed")

            us_rope = time_loop(torch, rope_steps, n_steps) / n_steps * 1e3
            res[w.name]["step_latency_us_rope"] = us_rope
            res[w.name]["frac_of_peak_rope"] = step_bytes / (us_rope * 1e-6) / 1e9 / peak
            del table
        cache.close()
        del blocks, ob
    # the 7 context blocks of the autoregressive 480p layer in one prefill call: block by block, and all together
    w = synth.AR480
    q, k, v = (torch.from_numpy(x.view("int16")).to(dev).view(torch.bfloat16) for x in synth.qkv(w))
    o = torch.empty_like(q)
    for name, nb in (("block_by_block", 0), ("all_blocks_together", w.n_blocks)):
        cache = la.BlockLinCache(w.B, w.H, w.d, torch.bfloat16, dev, max_T_b=w.T_b, eps=w.eps, prefill_blocks=nb)
        for _ in range(3):
            cache.prefill(q, k, v, w.n_blocks, out=o)
        n = 20
        ms = time_loop(torch, lambda i: cache.prefill(q, k, v, w.n_blocks, out=o), n) / n
        res.setdefault(w.name + "_prefill", {"blocks": w.n_blocks, "tokens": w.N,
                                             "l2": "one 257 MB input set (> 126 MB L2)"})[name + "_us"] = ms * 1e3
        cache.close()
    del q, k, v, o
    # temporal convolution of the Mix-FFN: the 480p / 720p layers, and block steps (3 frames) with the one-frame cache
    for wl in (synth.CONV_P480, synth.CONV_P720):
        x = torch.from_numpy(synth.conv_frames(wl).view("int16")).to(dev).view(torch.bfloat16)
        taps = torch.from_numpy(synth.conv_taps(wl.D, wl.seed)).to(dev)
        sets = [(x, torch.empty_like(x)), (x.flip(1).contiguous(), torch.empty_like(x))]
        for i in range(3):
            la.tconv_forward(sets[i & 1][0], taps, out=sets[i & 1][1])
        n = 20
        ms = time_loop(torch, lambda i: la.tconv_forward(sets[i & 1][0], taps, out=sets[i & 1][1]), n) / n
        by = 2 * x.numel() * 2
        res[wl.name] = {"B": wl.B, "frames": wl.T, "positions": wl.HW, "channels": wl.D, "ms": ms,
                        "algorithmic_gbs": by / (ms * 1e-3) / 1e9, "frac_of_peak": by / (ms * 1e-3) / 1e9 / peak,
                        "l2": "two rotating sets of %.0f MB (x and y) each" % (by / 1e6)}
        # block steps over the same frames: T_b = 3, blocks cycled so that every step's frames come from HBM
        n_blk = wl.T // 3
        cache = la.TConvCache(wl.B, wl.HW, wl.D, torch.bfloat16, dev)
        xs, ys = sets[0]
        for i in range(3):
            cache.step(xs[:, 3 * i:3 * i + 3], taps, out=ys[:, 3 * i:3 * i + 3])
        # the C entry point called with prebuilt descriptors and pointers, so that the host side of a step stays
        # well below the ~15 us the device needs
        import ctypes
        lib = la.load_library()
        desc = la._ConvDesc(wl.B, wl.HW, wl.D, la.LINATTN_BF16, xs.stride(0), ys.stride(0))
        blk_bytes = 3 * wl.HW * wl.D * 2
        calls = [(ctypes.c_void_p(xs.data_ptr() + j * blk_bytes), ctypes.c_void_p(ys.data_ptr() + j * blk_bytes))
                 for j in range(n_blk)]
        wp, cp = ctypes.c_void_p(taps.data_ptr()), ctypes.c_void_p(cache.frame.data_ptr())
        stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

        def step(i):
            xb, yb = calls[i % n_blk]
            if lib.tconv_block_step(ctypes.byref(desc), 3, xb, wp, cp, yb, 1, stream) != 0:
                raise RuntimeError("tconv_block_step failed")

        n = 4 * n_blk
        ms = time_loop(torch, step, n) / n
        by = (2 * 3 + 2) * wl.B * wl.HW * wl.D * 2      # 3 frames in and out, the cache frame read and written
        res[wl.name + "_block_step"] = {"frames_per_block": 3, "step_latency_us": ms * 1e3,
                                        "cache_bytes": cache.frame.numel() * 2,
                                        "algorithmic_gbs": by / (ms * 1e-3) / 1e9, "frac_of_peak": by / (ms * 1e-3) / 1e9 / peak,
                                        "l2": "%d blocks of one %.0f MB tensor pair cycled" % (n_blk, 4 * x.numel() / 1e6)}
        del x, sets, xs, ys, cache
    # the 720p bidirectional layer and its head-dim sweep at (about) the same width
    for w in (synth.P720, synth.p720_sweep(32), synth.p720_sweep(64), synth.p720_sweep(128)):
        q, k, v = (torch.from_numpy(x.view("int16")).to(dev).view(torch.bfloat16) for x in synth.qkv(w))
        o = torch.empty_like(q)
        ws = la.new_workspace(q)
        for _ in range(3):
            la.linattn_forward(q, k, v, w.eps, out=o, workspace=ws)
        n = 20
        ms = time_loop(torch, lambda i: la.linattn_forward(q, k, v, w.eps, out=o, workspace=ws), n) / n
        by = w.B * w.N * w.H * 8 * w.d
        res[w.name] = {"H": w.H, "d": w.d, "ms": ms, "tokens_heads_per_s": w.B * w.N * w.H / (ms * 1e-3),
                       "algorithmic_gbs": by / (ms * 1e-3) / 1e9, "frac_of_peak": by / (ms * 1e-3) / 1e9 / peak,
                       "l2": "one input set of %.0f MB (> 126 MB L2)" % (by / 1e6)}
        # the same layer with the rotary factors of Eq. 2 (3D table over the 21 x 45 x 80 latent grid)
        cos, sin = synth.rope_table(21, 45, 80, w.d)
        table = la.rope_pack(torch.from_numpy(cos).to(dev), torch.from_numpy(sin).to(dev))
        wsr = la.new_rope_workspace(q)
        for _ in range(3):
            la.linattn_forward_rope(q, k, v, table, w.eps, out=o, workspace=wsr)
        ms = time_loop(torch, lambda i: la.linattn_forward_rope(q, k, v, table, w.eps, out=o, workspace=wsr), n) / n
        res[w.name + "_rope"] = {"H": w.H, "d": w.d, "ms": ms, "tokens_heads_per_s": w.B * w.N * w.H / (ms * 1e-3),
                                 "algorithmic_gbs": by / (ms * 1e-3) / 1e9, "frac_of_peak": by / (ms * 1e-3) / 1e9 / peak,
                                 "note": "q,k,v,o bytes only; the fp16 rotation table (%.1f MB) is re-read from L2 by every "
                                         "tensor-core operand" % (table.numel() * 2 / 1e6)}
        del table, wsr, cos, sin
        if w.d == 112:
            # the same layer with head-major memory ([B,H,N,d] behind the same [B,N,H,d] view): a head's rows are
            # then contiguous instead of 224 bytes out of every 4480
            hm = lambda t: t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)
            qh, kh, vh = hm(q), hm(k), hm(v)
            oh = hm(o)
            wsh = la.new_workspace(qh)
            for _ in range(3):
                la.linattn_forward(qh, kh, vh, w.eps, out=oh, workspace=wsh)
            ms = time_loop(torch, lambda i: la.linattn_forward(qh, kh, vh, w.eps, out=oh, workspace=wsh), n) / n
            res[w.name + "_head_major"] = {"H": w.H, "d": w.d, "ms": ms, "layout": "[B,H,N,d] memory (strides in the descriptor)",
                                           "algorithmic_gbs": by / (ms * 1e-3) / 1e9, "frac_of_peak": by / (ms * 1e-3) / 1e9 / peak}
            del qh, kh, vh, oh, wsh
        del q, k, v, o, ws
    # Eq. 2 with its rotary factors on the 480p layer (3D table over the 21 x 30 x 52 latent grid)
    w = synth.P480
    q, k, v = (torch.from_numpy(x.view("int16")).to(dev).view(torch.bfloat16) for x in synth.qkv(w))
    cos, sin = synth.rope_table(21, 30, 52, w.d)
    table = la.rope_pack(torch.from_numpy(cos).to(dev), torch.from_numpy(sin).to(dev))
    outs = [torch.empty_like(q) for _ in range(2)]
    ins = [(q, k, v), (q.flip(1).contiguous(), k.flip(1).contiguous(), v.flip(1).contiguous())]
    wsr = la.new_rope_workspace(q)
    for i in range(3):
        la.linattn_forward_rope(*ins[i & 1], table, w.eps, out=outs[i & 1], workspace=wsr)
    n = 20
    ms = time_loop(torch, lambda i: la.linattn_forward_rope(*ins[i & 1], table, w.eps, out=outs[i & 1], workspace=wsr), n) / n
    by = w.B * w.N * w.H * 8 * w.d
    res[w.name + "_rope"] = {"H": w.H, "d": w.d, "ms": ms, "tokens_heads_per_s": w.B * w.N * w.H / (ms * 1e-3),
                             "algorithmic_gbs": by / (ms * 1e-3) / 1e9, "frac_of_peak": by / (ms * 1e-3) / 1e9 / peak,
                             "note": "q,k,v,o bytes only; the 7.3 MB fp16 rotation table is re-read from L2 by every head",
                             "l2": "two rotating input sets of 587 MB each"}
    return res


if __name__ == "__main__":
    main()

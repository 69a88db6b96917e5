"""Benchmark of preference-packed attention (plan + forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config NAME]

A step is one pass of the whole hot path over one synthetic batch: build the plan on the
device from the segment descriptors, forward (O, LSE), backward (Delta preprocess, main
kernel, dQ finalize).  The metric is useful TFLOP/s: 14 * Hq * D FLOPs per visible
(query, key) pair (2 GEMMs forward, 5 backward), masked pairs inside executed tiles not
counted.

Without --config the run covers every target workload -- configs[1], [2], [3] and the six
sweep points of configs[4] -- each with its own step time, kernel rooflines, clocks and
unpacked-pairs baseline under `per_config`; the top-level `value` is the largest workload (a
configs[4] point) and carries the end-to-end and CPU legs.  With --config only that workload
is measured.  Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "packed_attn_fwd_bwd_useful_tflops"
UNIT = "TFLOP/s"
NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_BF16_TFLOPS = 1590.0
TARGET_CONFIGS = ["config1", "config2", "config3"] + [f"config4:{i}" for i in range(6)]
HEADLINE = "config4:2"     # rho = 4, n = 2: the most useful FLOPs per step of all workloads

# Paper figures (end-to-end training ratios on unnamed hardware): context only.
PAPER_CONTEXT = {
    "training_time_reduction_at_least": 0.37,
    "speedup_with_batch_sorting": 3.22,
    "hardware": "a single GPU (model not stated) / multi-node FSDP (GPUs not stated)",
}


def get_workload(name: str, rank: int = 0):
    from paper_2602_24082_b200 import workloads as W
    if name == "config0":
        return W.config0()
    from paper_2602_24082_b200 import multi
    if name == "config1":
        return W.config1(seed=multi.rank_seed(1, rank))
    if name == "config2":
        return W.config2(seed=multi.rank_seed(2, rank, 10))
    if name == "config3":
        return W.config3(seed=multi.rank_seed(3, rank, 10))
    if name.startswith("config4"):
        point = int(name.split(":")[1]) if ":" in name else 0
        return W.config4(point)
    raise SystemExit(f"unknown config {name}")


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return (float(d["bf16_tflops"]), float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                float(d.get("hbm_gbs", 6650.0)), "measured")
    return FALLBACK_BF16_TFLOPS, 1400.0, 6650.0, "fallback"


def dram_traffic(config: str):
    """DRAM bytes per launch of the backward main kernel (dram__bytes_read.sum +
    dram__bytes_write.sum of one ncu capture), from the tracked summary
    profiles/bwd_kernel_dram_traffic.json: measured where a capture exists, otherwise scaled
    from the nearest captured workload by backward iterations, and labelled so."""
    path = os.path.join(ROOT, "profiles", "bwd_kernel_dram_traffic.json")
    if not os.path.exists(path):
        return None, "no capture"
    d = json.load(open(path)).get(config)
    if not d:
        return None, "no capture"
    return float(d["bytes"]), d.get("how", "ncu capture")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                try:
                    r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                except Exception:
                    r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def oracle_sample(w, tens, target_pairs: float = 2.0e8):
    """A bounded, independent sub-problem of the workload for the CPU oracle: whole groups,
    largest first among those that still fit, of one KV-head group, until about `target_pairs`
    visible pairs x query heads; more KV heads of the same groups when everything fits."""
    from paper_2602_24082_b200 import workloads as W
    r = w.num_q_heads // w.num_kv_heads
    pairs_of = lambda p, rs: p * (p + 1) // 2 + sum(x * p + x * (x + 1) // 2 for x in rs)
    groups = sorted(((pairs_of(p, rs) * r, ri, gi) for ri, row in enumerate(w.rows)
                     for gi, (p, rs) in enumerate(row)), reverse=True)
    picked, pairs = [], 0
    for (u, ri, gi) in groups:
        if pairs + u <= target_pairs or (not picked and u == groups[-1][0]):
            picked.append((ri, gi))
            pairs += u
    picked.sort()
    nkv = 1
    if len(picked) == len(groups):
        nkv = int(max(1, min(w.num_kv_heads, target_pairs // max(pairs, 1))))
    sub, stens, _, _ = W.slice_groups(w, tens, picked, list(range(nkv)))
    sizes = [w.rows[ri][gi][0] + sum(w.rows[ri][gi][1]) for ri, gi in picked]
    return sub, stens, (f"{len(picked)} of {len(groups)} groups (tokens {sizes[:8]}"
                        f"{' ...' if len(sizes) > 8 else ''}), KV heads 0..{nkv - 1} with their "
                        f"{r * nkv} query heads, {sub.useful_pairs() * r * nkv} pair-heads")


def time_oracle(sub, stens):
    import oracle
    t0 = time.perf_counter()
    oracle.attn_fwd_bwd(sub.descriptors(), *stens, sub.softmax_scale)
    dt = time.perf_counter() - t0
    f, b = sub.useful_flops()
    return (f + b) / dt / 1e12, dt, oracle.max_threads()


def workload_config(w, name, **extra):
    cfg = {
        "workload": f"{name}: {w.name}, {len(w.rows)} rows, T={w.total_tokens} tokens, "
                    f"Hq={w.num_q_heads}, Hkv={w.num_kv_heads}, D={w.head_dim}, "
                    f"visible pairs U={w.useful_pairs()}",
        "step": "pp_build_plan + pp_attn_fwd + pp_attn_bwd",
        "l2": "flushed between timed steps (512 MiB write)",
        "per_gpu_batch": "one batch of the recipe per GPU (seed differs per rank)",
    }
    cfg.update(extra)
    return cfg


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    name = args.config or HEADLINE
    w = get_workload(name, 0)
    tens = w.tensors()
    sub, stens, what = oracle_sample(w, tens, target_pairs=5.0e7)
    import oracle
    oracle.build()
    for _ in range(min(args.warmup, 1)):
        time_oracle(sub, stens)
    times, cores = [], 1
    for _ in range(args.steps):
        _, dt, cores = time_oracle(sub, stens)
        times.append(dt)
    f, b = sub.useful_flops()
    value = (f + b) * len(times) / sum(times) / 1e12
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * sum(times) / len(times),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": workload_config(w, name),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": what},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


class Runner:
    """Measures one workload on the current device."""

    def __init__(self, args, rank, world, local):
        import torch
        self.torch = torch
        self.args, self.rank, self.world, self.local = args, rank, world, local
        self.dev = f"cuda:{local}"
        self.flush = torch.empty(512 << 20, dtype=torch.uint8, device=self.dev)
        self.peak, self.peak_sustained, self.hbm, self.peak_kind = peaks()

    def barrier(self):
        if self.world > 1:
            import torch.distributed as dist
            dist.barrier()
        self.torch.cuda.synchronize()

    def timed(self, fn, steps, profile=False):
        """`steps` calls of fn, each behind an L2 flush and bracketed by CUDA events on the
        current stream.  Returns (ms per call, per-call kernel event readings, launches)."""
        from paper_2602_24082_b200 import binding as B
        torch = self.torch
        evs, kern, launches = [], [], 0
        for _ in range(steps):
            self.flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            launches += fn() or 0
            e1.record()
            evs.append((e0, e1))
        torch.cuda.synchronize()
        if profile:
            # the library keeps a ring of event pairs per kernel: no synchronisation between the
            # timed steps (it would expose the host's launch latency inside the timed region)
            fk, bk = B.pp_profile_read_all(64)
            n = min(steps, 64)
            bk = bk[-n:]
            fk = fk[-n:] if fk else [None] * len(bk)
            kern = list(zip(fk, bk))
        return [a.elapsed_time(b) for a, b in evs], kern, launches

    def measure(self, name, w, headline: bool):
        import numpy as np
        torch = self.torch
        from paper_2602_24082_b200 import binding as B
        from paper_2602_24082_b200 import workloads as W
        from paper_2602_24082_b200 import cost_model
        from paper_2602_24082_b200 import multi
        args, dev = self.args, self.dev
        steps = args.steps if headline else max(3, min(args.steps, 20))
        warmup = max(args.warmup, 3)

        tens_cpu = w.tensors()
        q, k, v, do = (x.to(dev) for x in tens_cpu)
        if not headline:
            del tens_cpu
        desc = w.descriptors()
        desc_dev = [torch.from_numpy(np.ascontiguousarray(a)).to(dev) for a in desc]
        T, Hq, Hkv, D = w.total_tokens, w.num_q_heads, w.num_kv_heads, w.head_dim
        problem, _keep = B.make_problem(desc, Hq, Hkv, D, T, desc_dev)
        plan_bytes, _, bwd_bytes = B.pp_plan_workspace_bytes(problem)
        ws = torch.empty(plan_bytes, dtype=torch.uint8, device=dev)
        scratch = torch.empty(bwd_bytes, dtype=torch.uint8, device=dev)
        o = torch.empty_like(q)
        lse = torch.empty(Hq, T, dtype=torch.float32, device=dev)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        scale = w.softmax_scale
        hold = {}

        def step():
            plan = B.pp_build_plan(desc, Hq, Hkv, D, T, dev, device_arrays=desc_dev, workspace=ws)
            n = B.pp_last_launch_count()
            plan._bwd_scratch = scratch
            B.pp_attn_fwd(plan, q, k, v, scale, o=o, lse=lse, for_backward=True)
            n += B.pp_last_launch_count()
            B.pp_attn_bwd(plan, q, k, v, o, lse, do, scale, d_q=dq, d_k=dk, d_v=dv)
            n += B.pp_last_launch_count()
            hold["plan"] = plan
            return n

        for _ in range(warmup):
            self.flush.zero_()
            step()
        torch.cuda.synchronize()
        st = hold["plan"].status()
        if st != (0, 0):
            raise SystemExit(f"{name}: device status {st}")

        # Kernel timing inside the timed region: events around the backward main kernel only
        # (the kernel the roofline is for); an event between two kernels keeps the second from
        # being queued behind the first, so the forward kernel is timed in a short pass of its
        # own directly before.
        B.pp_profile_enable(True)
        _, kern_f, _ = self.timed(step, min(steps, 10), profile=True)
        fwd_ms = statistics.mean(x[0] for x in kern_f)
        B.pp_profile_enable(True, backward_only=True)
        sampler = ClockSampler(self.local)
        self.barrier()
        sampler.start()
        ms, kern, launches = self.timed(step, steps, profile=True)
        self.barrier()
        clocks = sampler.stop()
        B.pp_profile_enable(False)
        f_flops, b_flops = w.useful_flops()
        # max over ranks of the timed region; sum over ranks of the work (one batch per rank)
        total_ms, flops_all, tokens_all = multi.aggregate(sum(ms), float(f_flops + b_flops), float(T), dev)
        ms_per_step = total_ms / steps
        value = multi.whole_job_throughput(total_ms, steps, flops_all)

        bwd_ms = statistics.mean(x[1] for x in kern)
        bwd_tflops = b_flops / (bwd_ms * 1e-3) / 1e12
        fwd_tflops = f_flops / (fwd_ms * 1e-3) / 1e12
        # steps of a few ms and more run under the power cap: the sustained peak is the fair one
        long_step = ms_per_step >= 5.0
        peak_used = self.peak_sustained if long_step else self.peak
        traffic, traffic_how = dram_traffic(name)
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "steps": steps, "warmup": warmup,
            "ms_per_step": ms_per_step, "ms_min_median": [min(ms), statistics.median(ms)],
            "config": workload_config(w, name),
            "clocks": clocks,
            "gpu_launches": launches,
            "tokens_per_s": tokens_all / (ms_per_step * 1e-3),
            "pct_of_peak": {"measured_burst": 100 * value / self.peak,
                            "measured_sustained": 100 * value / self.peak_sustained,
                            "nominal": 100 * value / NOMINAL_BF16_TFLOPS},
            "roofline": {"kernel": "bwd_kernel (dS/dQ/dK/dV main)", "bound": "tensor",
                         "achieved": bwd_tflops, "peak": peak_used, "unit": "TFLOP/s",
                         "frac": bwd_tflops / peak_used,
                         "peak_kind": f"of {self.peak_kind} ({'sustained' if long_step else 'burst'})",
                         "frac_of_burst_peak": bwd_tflops / self.peak,
                         "frac_of_sustained_peak": bwd_tflops / self.peak_sustained,
                         "traffic": traffic, "traffic_source": traffic_how,
                         "traffic_unit": "bytes (dram read + write per launch)",
                         "algorithmic_flops_per_launch": float(b_flops), "avg_launch_ms": bwd_ms},
            "roofline_fwd": {"kernel": "fwd_kernel", "bound": "tensor", "achieved": fwd_tflops,
                             "peak": peak_used, "unit": "TFLOP/s", "frac": fwd_tflops / peak_used,
                             "frac_of_burst_peak": fwd_tflops / self.peak, "avg_launch_ms": fwd_ms,
                             "note": "timed in a separate pass directly before the timed region"},
            "outside_main_kernels_ms": ms_per_step - fwd_ms - bwd_ms,
        }

        if self.world == 1 and not args.quick:
            # ---- the same kernels on the unpacked paired batch (each [x, y_k] its own sequence)
            base = statistics.median(ms)
            for padded in (True, False):
                uw, gather = W.unpacked(w, padded=padded)
                g = gather.to(dev)
                uq, uk, uv, udo = (x.index_select(0, g).contiguous() for x in (q, k, v, do))
                uplan = B.plan_for(uw, dev, desc_on_device=True)
                uo, ulse = B.pp_attn_fwd(uplan, uq, uk, uv, scale)
                B.pp_attn_bwd(uplan, uq, uk, uv, uo, ulse, udo, scale)

                def ustep():
                    pl = B.pp_build_plan(uw.descriptors(), Hq, Hkv, D, uw.total_tokens, dev,
                                         device_arrays=uplan._keep[1], workspace=uplan.workspace)
                    pl._bwd_scratch = uplan.bwd_scratch()
                    B.pp_attn_fwd(pl, uq, uk, uv, scale, o=uo, lse=ulse, for_backward=True)
                    B.pp_attn_bwd(pl, uq, uk, uv, uo, ulse, udo, scale)
                    return 0

                for _ in range(2):
                    ustep()
                ums, _, _ = self.timed(ustep, max(3, min(steps, 8)))
                key = "unpacked_padded" if padded else "unpacked_unpadded"
                out[key] = {"ms_per_step": statistics.median(ums), "tokens": uw.total_tokens,
                            "speedup_of_packed": statistics.median(ums) / base,
                            "useful_pair_ratio": uw.useful_pairs() / w.useful_pairs()}
                del uq, uk, uv, udo, uo, ulse, uplan
            grp = [(p, rs) for row in w.rows for (p, rs) in row]
            out["paper_cost_model_mean"] = {
                "attention_cost_ratio": statistics.mean(cost_model.attention_cost_ratio(p, rs) for p, rs in grp),
                "memory_ratio": statistics.mean(cost_model.memory_ratio(p, rs) for p, rs in grp)}

        if headline:
            self.headline_extras(out, w, name, tens_cpu, step, hold, (q, k, v, do, o, lse, dq, dk, dv),
                                 flops_all, steps)
        return out

    def headline_extras(self, out, w, name, tens_cpu, step, hold, tensors, flops_all, steps):
        """End-to-end leg through host buffers, the rows beyond the attention kernels, the step
        without kernel events and as a CUDA graph, and the CPU oracle beside it."""
        import numpy as np
        torch = self.torch
        from paper_2602_24082_b200 import binding as B
        from paper_2602_24082_b200 import multi
        q, k, v, do, o, lse, dq, dk, dv = tensors
        dev, args = self.dev, self.args
        T, Hq, Hkv, D = w.total_tokens, w.num_q_heads, w.num_kv_heads, w.head_dim
        scale = w.softmax_scale
        f_flops, b_flops = w.useful_flops()

        # ---- end to end through pp_attn_step_host: pinned host buffers, copies inside the timing
        host = B.HostStep(w, dev)
        hq, hk, hv, hdo = (x.pin_memory() for x in tens_cpu)
        for _ in range(2):
            host(hq, hk, hv, hdo)
        torch.cuda.synchronize()
        self.barrier()
        e2e_ms, _, _ = self.timed(lambda: host(hq, hk, hv, hdo) and 0, max(3, min(steps, 8)))
        self.barrier()
        e2e_total, _, _ = multi.aggregate(sum(e2e_ms) / len(e2e_ms), 0.0, 0.0, dev)
        out["e2e"] = {"value": flops_all / (e2e_total * 1e-3) / 1e12, "unit": UNIT,
                      "h2d_bytes_per_step": host.h2d_bytes, "d2h_bytes_per_step": host.d2h_bytes,
                      "ms_per_step": e2e_total, "api": "pp_attn_step_host (pinned host buffers)"}
        del host, hq, hk, hv, hdo
        if self.world > 1 or self.rank != 0:
            return

        plan = hold["plan"]
        # ---- next row of the path: packed position ids + rotary embedding on Q/K (HBM-bound)
        rq, rk = q.clone(), k.clone()
        for _ in range(3):
            B.pp_rope_qk(plan, rq, rk, 500000.0)
        rms, _, _ = self.timed(lambda: (B.pp_rope_qk(plan, rq, rk, 500000.0), 0)[1], 10)
        rbytes = 2.0 * 2.0 * T * (Hq + Hkv) * D
        gbs = rbytes / (statistics.median(rms) * 1e-3) / 1e9
        out["rope_qk"] = {"ms": statistics.median(rms), "bytes": rbytes,
                          "roofline": {"bound": "hbm", "achieved": gbs, "peak": self.hbm, "unit": "GB/s",
                                       "frac": gbs / self.hbm}}
        del rq, rk
        # ---- next row: loss-side consumer (per-response log-probs + pairwise preference loss)
        tl = -torch.rand(T, device=dev) * 3
        tr = -torch.rand(T, device=dev) * 3
        for _ in range(3):
            B.pp_preference_loss(plan, tl, tr, 0.1)
        lms, _, _ = self.timed(lambda: (B.pp_preference_loss(plan, tl, tr, 0.1), 0)[1], 10)
        lbytes = 12.0 * T
        lg = lbytes / (statistics.median(lms) * 1e-3) / 1e9
        out["preference_loss"] = {"ms": statistics.median(lms), "bytes": lbytes,
                                  "note": "latency-bound: one warp per group, 12 bytes per token",
                                  "roofline": {"bound": "hbm", "achieved": lg, "peak": self.hbm,
                                               "unit": "GB/s", "frac": lg / self.hbm}}

        # ---- next row: the bit-reproducible backward (key tiles add to dQ in turn)
        B.pp_profile_enable(True)
        B.pp_attn_fwd(plan, q, k, v, scale, o=o, lse=lse)   # (both event pairs must be valid)
        dms, nms = [], []
        for det in (True, False, True, False):
            for _ in range(4):
                self.flush.zero_()
                B.pp_attn_bwd(plan, q, k, v, o, lse, do, scale, d_q=dq, d_k=dk, d_v=dv,
                              deterministic=det)
                torch.cuda.synchronize()
                (dms if det else nms).append(B.pp_profile_read()[1])
        B.pp_profile_enable(False)
        out["deterministic_bwd"] = {
            "main_kernel_ms": statistics.median(dms), "default_main_kernel_ms": statistics.median(nms),
            "tflops": b_flops / (statistics.median(dms) * 1e-3) / 1e12,
            "slowdown": statistics.median(dms) / statistics.median(nms)}

        # ---- next row: head_dim 96 (the same packing structure and head counts; the kernels run
        # it in tiles of 128 columns whose upper quarter the TMA loads fill with zeros)
        from paper_2602_24082_b200 import workloads as W96
        w96 = W96.Workload(w.name + "-d96", w.rows, Hq, Hkv, 96, seed=96)
        q9, k9, v9, do9 = (x.to(dev) for x in w96.tensors())
        plan9 = B.plan_for(w96, desc_on_device=True)
        f9, b9 = w96.useful_flops()
        o9 = lse9 = None
        for _ in range(3):
            o9, lse9 = B.pp_attn_fwd(plan9, q9, k9, v9, w96.softmax_scale)
            B.pp_attn_bwd(plan9, q9, k9, v9, o9, lse9, do9, w96.softmax_scale)
        fms, bms = [], []
        for _ in range(5):
            self.flush.zero_()
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
            ev[0].record()
            o9, lse9 = B.pp_attn_fwd(plan9, q9, k9, v9, w96.softmax_scale)
            ev[1].record()
            B.pp_attn_bwd(plan9, q9, k9, v9, o9, lse9, do9, w96.softmax_scale)
            ev[2].record()
            torch.cuda.synchronize()
            fms.append(ev[0].elapsed_time(ev[1]))
            bms.append(ev[1].elapsed_time(ev[2]))
        fm, bm = statistics.median(fms), statistics.median(bms)
        out["head_dim_96"] = {"fwd_ms": fm, "bwd_ms": bm,
                              "fwd_tflops": f9 / (fm * 1e-3) / 1e12,
                              "bwd_tflops": b9 / (bm * 1e-3) / 1e12,
                              "value": (f9 + b9) / ((fm + bm) * 1e-3) / 1e12, "unit": "TFLOP/s",
                              "note": "forward + backward (preprocess, main, finalize), plan excluded"}
        del q9, k9, v9, do9, o9, lse9, plan9

        # ---- next row: the row builder (batch sorting + packing into rows) on a synthetic
        # batch of 4096 preference groups of up to 16K tokens, rows of 16384 tokens, and the
        # assignment of those rows to 8 data-parallel ranks
        rng = np.random.default_rng(17)
        gP = rng.integers(64, 8000, size=4096).astype(np.int32)
        goff = (np.arange(4097) * 2).astype(np.int32)
        grl = rng.integers(16, 4000, size=8192).astype(np.int32)
        dP, doff, drl = (torch.from_numpy(a).to(dev) for a in (gP, goff, grl))
        for _ in range(3):
            rb = B.pp_build_rows(dP, doff, drl, 16384)
        bms, _, _ = self.timed(lambda: (B.pp_build_rows(dP, doff, drl, 16384), 0)[1], 10)
        out["row_builder"] = {"ms": statistics.median(bms), "groups": 4096,
                              "rows": int(rb["row_group_off"].numel()) - 1, "row_capacity": 16384,
                              "tokens": int(rb["row_tokens"].sum().item()),
                              "note": "integer work in three small kernels; the time includes the "
                                      "binding's allocations and its status read-back"}
        for _ in range(3):
            ar = B.pp_assign_rows(rb["row_cost"], 8)
        ams, _, _ = self.timed(lambda: (B.pp_assign_rows(rb["row_cost"], 8), 0)[1], 10)
        rc = ar[2].double()
        out["row_assignment"] = {"ms": statistics.median(ams), "rows": int(rb["row_cost"].numel()),
                                 "ranks": 8, "max_over_mean_rank_cost": float(rc.max() / rc.mean())}

        # ---- the same step without any event between its kernels: as plain stream launches
        # and captured once in a CUDA graph and replayed
        ems, _, _ = self.timed(step, min(steps, 30))
        emed = statistics.median(ems)
        out["no_kernel_events"] = {"ms_per_step": emed, "value": (f_flops + b_flops) / (emed * 1e-3) / 1e12,
                                   "unit": UNIT, "note": "median of per-step times"}
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                step()
            for _ in range(3):
                graph.replay()
            gms, _, _ = self.timed(lambda: (graph.replay(), 0)[1], min(steps, 30))
            gmed = statistics.median(gms)
            out["graph_replay"] = {"ms_per_step": gmed, "value": (f_flops + b_flops) / (gmed * 1e-3) / 1e12,
                                   "unit": UNIT,
                                   "note": "plan + forward + backward captured in one CUDA graph"}
            del graph
        except Exception as e:   # a convenience figure, not part of the measured path
            out["graph_replay"] = {"unavailable": str(e)[:200]}

        # ---- the CPU oracle beside it (rank 0, N = 1 only), on a bounded sample
        if not args.no_cpu_baseline:
            sub, stens, what = oracle_sample(w, tens_cpu, target_pairs=args.cpu_pairs)
            v_cpu, dt, cores = time_oracle(sub, stens)
            out["cpu_baseline"] = {"value": v_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                                   "sample": what + f"; {dt:.1f} s"}


def rank_workload(name, rank, world, dev):
    """The batch a rank processes.  One GPU: the recipe's batch.  Several GPUs (data parallel,
    no exchange inside the path): the ranks' batches are pooled and the rows are dealt out by
    attention cost with pp_assign_rows -- every rank computes the same assignment on its own
    GPU from the same costs -- so that no rank waits for the one with the longest rows."""
    if world == 1:
        return get_workload(name, rank), None
    import torch
    from paper_2602_24082_b200 import binding as B
    from paper_2602_24082_b200 import multi
    batches = [get_workload(name, r) for r in range(world)]
    pool, costs = multi.pool_rows(batches)
    _, rank_of_row, rank_cost = B.pp_assign_rows(torch.tensor(costs, dtype=torch.int64, device=dev), world)
    w = multi.rank_batch(batches, pool, rank_of_row.tolist(), rank)
    rc = rank_cost.double()
    return w, {"rows_pooled": len(pool), "assignment": "pp_assign_rows (longest cost first)",
               "max_over_mean_rank_cost": float(rc.max() / rc.mean())}


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2602_24082_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))
    B.lib()
    runner = Runner(args, rank, world, local)

    head_name = args.config or HEADLINE
    others = [] if (args.config or world > 1 or args.quick) else [c for c in TARGET_CONFIGS if c != head_name]
    per_config = {}
    for name in others:
        w = get_workload(name, rank)
        per_config[name] = runner.measure(name, w, headline=False)
        torch.cuda.empty_cache()

    w, dp = rank_workload(head_name, rank, world, dev)
    if args.quick:
        args.no_cpu_baseline = True
    head = runner.measure(head_name, w, headline=not args.quick)
    if rank == 0:
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": head["steps"],
            "warmup": head["warmup"], "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        }
        for k_, v_ in head.items():
            if k_ not in line:
                line[k_] = v_
        if dp:
            line["data_parallel"] = dp
        line.setdefault("cpu_baseline", None)
        line["paper_context"] = PAPER_CONTEXT
        if per_config:
            slim = lambda d: {k_: d[k_] for k_ in ("value", "unit", "ms_per_step", "steps", "clocks", "pct_of_peak",
                                                   "tokens_per_s", "roofline", "roofline_fwd",
                                                   "outside_main_kernels_ms", "unpacked_padded",
                                                   "unpacked_unpadded", "paper_cost_model_mean", "config")
                              if k_ in d}
            per_config[head_name] = head
            line["per_config"] = {n: slim(per_config[n]) for n in TARGET_CONFIGS if n in per_config}
            pct = {n: per_config[n]["pct_of_peak"] for n in line["per_config"]}
            line["min_pct_of_peak_over_configs"] = {
                kind: min(p[kind] for p in pct.values()) for kind in ("measured_burst", "measured_sustained", "nominal")}
            line["min_pct_of_peak_over_configs"]["config"] = min(pct, key=lambda n: pct[n]["measured_burst"])
            line["packed_faster_than_unpacked_on_every_config"] = all(
                per_config[n].get("unpacked_padded", {}).get("speedup_of_packed", 0) > 1.0 and
                per_config[n].get("unpacked_unpadded", {}).get("speedup_of_packed", 0) > 1.0
                for n in line["per_config"])
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=None,
                    help="measure only this workload (config1, config2, config3, config4:0..5)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-pairs", type=float, default=5.0e8,
                    help="size of the CPU oracle's sample in visible pairs x query heads")
    ap.add_argument("--quick", action="store_true",
                    help="timed steps only (no e2e, unpacked baseline or CPU leg): for profiler runs")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps == 20 and args.warmup == 5:
            args.steps, args.warmup = 3, 1
        run_reference(args)
        return
    if args.gpus > 1 and "RANK" not in os.environ:
        # started plainly: bring up one rank per GPU and let rank 0 print the line
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 2000),
               os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    run_ours(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the region-trace hot path: marker events/s for one pass of
pair -> aggregate -> overlap over one synthetic trace, and the HBM roofline fraction of the
dominant (pairing) kernel.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload I]

One process per GPU (torchrun for N > 1); every rank processes its own trace of the same shape
(weak scaling, no data-path collective). Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "marker events/sec (pair+aggregate, 1 B200) and % of HBM roofline"  # the step also runs the overlap stage
UNIT = "events/s"
ALG_BYTES_PER_EVENT = 40.0  # 16 B event read + 48 B interval written per 2 events
# DRAM traffic of the pairing kernel from one ncu capture (dram__bytes_read.sum + dram__bytes_write.sum of one launch)
# on a small case of the bench workload; the full trace is too large for a multi-pass capture, and the kernel's
# traffic grows in proportion to the events, so the JSON line scales it to a full launch and says so.
TRAFFIC_CAPTURE = {"workload": "decode_megakernel", "iters": 8, "events": 38380544, "dram_bytes_read": 614.345216e6,
                   "dram_bytes_write": 1019.052e6, "kernel": "k_pair_tiled<128,5,7>",
                   "command": "ncu --set full --clock-control none -k regex:k_pair_tiled -s 6 -c 1 python bench.py --workload 3 "
                              "--iters 8 --steps 1 --warmup 3 --no-e2e --no-cpu-baseline --no-other"}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock, power and clock-event reasons of one GPU through NVML while running."""
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting", 0x10: "sync_boost"}

    def __init__(self, torch_device):
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            props = torch.cuda.get_device_properties(torch_device)
            h = None
            uuid = getattr(props, "uuid", None)
            if uuid is not None:
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
                except Exception:
                    try:
                        h = pynvml.nvmlDeviceGetHandleByUUID("GPU-" + str(uuid))
                    except Exception:
                        h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(torch_device.index or 0)
            self._h = h
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML missing: report that clocks were not sampled
            self.error = repr(e)

    def _loop(self):
        nv, h = self._nv, self._h
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
                self.power.append(nv.nvmlDeviceGetPowerUsage(h) / 1000.0)
            except Exception:
                pass
            time.sleep(0.005)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0,
                    "note": getattr(self, "error", "no samples")}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples), "power_w_max": max(self.power) if self.power else None}


def oracle_step(oracle, ev, offs, spec, cta_sm, num_sms):
    rc, iv, ioffs, am, aoffs, st = oracle.pair(ev, offs, spec.num_regions, ambig_cap=max(len(ev) // 64, 4096))
    assert rc == 0 and int(st["code"]) == 0
    rc, tabs, st = oracle.aggregate(iv, ioffs, am, aoffs, spec.warps_per_cta, cta_sm, num_sms, spec.num_regions)
    assert rc == 0
    rc, ov, st = oracle.overlap(iv, ioffs, spec.warps_per_cta, cta_sm, num_sms, spec.overlap_pairs)
    assert rc == 0
    return tabs, ov


def oracle_sample(tg, spec, num_ctas):
    """Host copy of the first `num_ctas` CTAs of the workload (bit-identical to the device trace)."""
    offs = tg.host_offsets(spec)
    num_ctas = min(num_ctas, spec.num_ctas)
    S = num_ctas * spec.warps_per_cta
    ev = tg.host_streams(spec, offs, 0, S)
    sub = (offs[: S + 1] - offs[0]).astype(np.uint64)
    cta_sm = spec.cta_sm[:num_ctas].copy()
    return ev, sub, cta_sm, int(cta_sm.max()) + 1


def run_reference(args, spec, tg):
    """The oracle as it stands, on the host cores, on a bounded sample of the workload per step."""
    import oracle
    oracle.build()
    num_ctas = 1
    ev, offs, cta_sm, num_sms = oracle_sample(tg, spec, num_ctas)
    for _ in range(args.warmup):
        oracle_step(oracle, ev, offs, spec, cta_sm, num_sms)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(oracle, ev, offs, spec, cta_sm, num_sms)
    dt = time.perf_counter() - t0
    value = len(ev) * args.steps / dt
    sample = f"first {num_ctas} CTA(s) = {num_ctas * spec.warps_per_cta} streams, {len(ev)} events per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64", "data": "synthetic",
        "config": {"workload": spec.name, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=3, help="config index 0..4 (default 3: decode megakernel, the largest)")
    ap.add_argument("--iters", type=int, default=0, help="override the workload's iteration count (smaller trace for profiler captures)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--cpu-ctas", type=int, default=6, help="CTAs of the workload the CPU baseline is timed on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--three-calls", action="store_true",
                    help="time argus_pair_intervals + argus_aggregate + argus_overlap instead of the one-call argus_synthesize")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-other", action="store_true",
                    help="skip the secondary records (three plain calls, corrupted marker, the other trace shapes)")
    ap.add_argument("--no-combine", action="store_true",
                    help="N > 1: do not combine the ranks' kernel-scope tables at the end of every step")
    ap.add_argument("--suite", default="main", choices=["main", "secondary"],
                    help="secondary: timings of the entry points beyond the step (bench_secondary.py), one JSON line each")
    ap.add_argument("--what", default="join", choices=["scoped", "pcmap", "ring", "join"], help="--suite secondary: which one")
    ap.add_argument("--queries", type=int, default=2000, help="--suite secondary --what join: number of queries")
    args = ap.parse_args()
    if args.suite == "secondary":
        import bench_secondary
        bench_secondary.run(args.what, iters=args.iters, queries=args.queries)
        return
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    from paper_2609_12299_b200.multirank import combine_kernel_tables, max_over_ranks, rank_env, rank_spec, whole_job_rate
    rank, world, local_rank = rank_env()

    from paper_2609_12299_b200 import tracegen as tg
    spec = tg.config(args.workload)
    if args.iters:
        spec = spec.scaled(iters=args.iters)

    if args.impl == "reference":
        if rank == 0:
            run_reference(args, spec, tg)
        return

    import torch
    import torch.distributed as dist

    import paper_2609_12299_b200 as argus

    argus.load_library()  # raises if the CUDA library was not built: there is no fallback
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device")
    dev = torch.device("cuda", local_rank)
    torch.cuda.set_device(dev)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    # every rank its own trace of the same shape (weak scaling)
    spec = rank_spec(spec, rank)
    d_ev, d_off = tg.generate_cuda(spec, dev)
    n_events = d_ev.numel() // 16
    S = spec.num_streams
    combine = world > 1 and not args.no_combine

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    class Runner:
        """One workload resident on the device: its step functions and their output buffers (allocated once)."""

        def __init__(self, spec, d_ev, d_off):
            self.spec, self.d_ev, self.d_off = spec, d_ev, d_off
            self.n = d_ev.numel() // 16
            self.cta_sm = torch.from_numpy(spec.cta_sm.view(np.int32)).to(dev)
            self.pairs = torch.from_numpy(spec.overlap_pairs.view(np.int32)).to(dev)
            self.icap = self.n // 2
            self.acap = max(self.n // 64, 4096)
            self.mos = max(self.n // 8, 1 << 16)  # overlap spans the one-call pipeline may select
            self.state = {"pair": None, "agg": None, "syn": None, "ov": None}
            self.ov_ws = None

        def step_three_calls(self):
            sp, st = self.spec, self.state
            if self.ov_ws is None:
                self.ov_ws = torch.empty(min(argus.argus_overlap_workspace_bytes(self.icap, sp.num_streams, len(sp.overlap_pairs),
                                                                                 sp.num_sms), 2 << 30), dtype=torch.uint8, device=dev)
            st["pair"] = p = argus.argus_pair_intervals(self.d_ev, self.d_off, sp.num_regions, interval_capacity=self.icap,
                                                        ambig_capacity=self.acap, out=st["pair"])
            st["agg"] = argus.argus_aggregate(p.intervals, p.interval_offsets, p.ambig, p.ambig_offsets, sp.warps_per_cta,
                                              self.cta_sm, sp.num_sms, sp.num_regions, out=st["agg"])
            st["ov"] = argus.argus_overlap(p.intervals, self.icap, p.interval_offsets, sp.warps_per_cta, self.cta_sm, sp.num_sms,
                                           self.pairs, workspace=self.ov_ws)

        def step_one_call(self):
            sp, st = self.spec, self.state
            st["syn"] = r = argus.argus_synthesize(self.d_ev, self.d_off, sp.num_regions, sp.warps_per_cta, self.cta_sm,
                                                   sp.num_sms, self.pairs, interval_capacity=self.icap, ambig_capacity=self.acap,
                                                   max_overlap_spans=self.mos, out=st["syn"])
            st["pair"], st["agg"], st["ov"] = r.pair, r.agg, (r.overlap, r.status)

        def check_status(self, where):
            for name in ("pair", "agg"):
                code = int(argus.argus_status_fetch(self.state[name].status)["code"])
                if code != 0:
                    raise RuntimeError(f"device status {code} in {name} {where}")
            if int(argus.argus_status_fetch(self.state["ov"][1])["code"]) != 0:
                raise RuntimeError(f"device status in overlap {where}")

        def timed(self, local_step, steps, warmup, exchange=False, sampler=None):
            """`warmup` untimed steps, then `steps` steps between CUDA events; kernel times from the library's own events."""
            def step():
                local_step()
                if exchange:  # the path's one exchange step: R x 576 bytes, all-reduced (sum / min / max)
                    combine_kernel_tables(self.state["agg"].kernel, world)
            for _ in range(warmup):
                step()
            barrier()
            self.check_status("after warm-up")
            argus.argus_profile_read()
            argus.argus_profile_enable(True)
            launches0 = argus.argus_launch_count()
            if sampler:
                sampler.start()
            barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(steps):
                step()
            e1.record()
            barrier()
            if sampler:
                sampler.stop()
            launches = argus.argus_launch_count() - launches0
            argus.argus_profile_enable(False)
            prof_ms, prof_n = argus.argus_profile_read()
            self.check_status("after the timed region")
            kernel_ms = {k: prof_ms[k] / max(prof_n[k], 1) for k in ("pair", "aggregate", "overlap")}
            return e0.elapsed_time(e1), launches, kernel_ms, step

    main_run = Runner(spec, d_ev, d_off)
    local_step = main_run.step_three_calls if args.three_calls else main_run.step_one_call
    sampler = ClockSampler(dev)
    ms_total, launches, kernel_ms, step = main_run.timed(local_step, args.steps, args.warmup, combine, sampler)
    state = main_run.state
    prof_pair_ms = kernel_ms["pair"]

    ms_total = max_over_ranks(ms_total, world, dev)
    ms_per_step = ms_total / args.steps
    value = whole_job_rate(n_events, world, ms_per_step)

    # roofline of the dominant kernel (the pairing kernel): algorithmic bytes / its own launch time
    peak, peak_src = load_peaks()
    pair_ms = prof_pair_ms
    achieved = ALG_BYTES_PER_EVENT * n_events / (pair_ms * 1e-3) / 1e9 if pair_ms > 0 else 0.0
    step_gbs = ALG_BYTES_PER_EVENT * n_events / (ms_per_step * 1e-3) / 1e9
    scaled = (TRAFFIC_CAPTURE["dram_bytes_read"] + TRAFFIC_CAPTURE["dram_bytes_write"]) / TRAFFIC_CAPTURE["events"] * n_events
    roofline = {"bound": "hbm", "kernel": "tiled pairing kernel (k_pair_tiled), the dominant kernel, timed alone",
                "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "frac_of_8TBs_nominal": achieved / 8000.0, "peak_source": peak_src,
                "traffic": scaled if spec.name == TRAFFIC_CAPTURE["workload"] else None,
                "traffic_source": "ncu capture of one launch on a smaller case of the same trace, scaled by events",
                "traffic_capture": TRAFFIC_CAPTURE,
                "ms_per_launch": pair_ms, "algorithmic_bytes_per_event": ALG_BYTES_PER_EVENT,
                # the whole step (every kernel of pair + aggregate + overlap) by the accounting of a fused pair + aggregate
                "step": {"achieved": step_gbs, "frac": step_gbs / peak, "frac_of_8TBs_nominal": step_gbs / 8000.0,
                         "ms": ms_per_step},
                "pipeline_frac": step_gbs / peak}
    if kernel_ms["aggregate"] > 0:
        # the pass over the intervals' digests (aggregation + overlap span selection): 8 B read per interval; it is
        # bound by instruction issue and shared-memory atomics, the HBM figure is given for scale
        agg_gbs = 4.0 * n_events / (kernel_ms["aggregate"] * 1e-3) / 1e9
        roofline["second_kernel"] = {"kernel": "per-stream aggregation pass over the digests (k_agg_streams_digest)",
                                     "bound": "issue / shared-memory atomics", "bytes_read_per_event": 4.0,
                                     "ms_per_launch": kernel_ms["aggregate"], "achieved": agg_gbs, "frac_of_hbm": agg_gbs / peak}

    # end to end with HOST buffers: pinned events -> device, the three calls, result tables -> host
    e2e = None
    if not args.no_e2e:
        pin_ev = torch.empty(n_events * 16, dtype=torch.uint8, pin_memory=True)
        pin_ev.copy_(d_ev)
        pin_off = torch.empty(S + 1, dtype=torch.int64, pin_memory=True)
        pin_off.copy_(d_off)
        agg = state["agg"]
        # tables, overlap, offsets and status come back; the interval array (48 B per interval) stays on the device
        outs = [agg.kernel, agg.sm, agg.cta, state["ov"][0], state["pair"].interval_offsets, state["pair"].status]
        pin_out = [torch.empty(o.numel(), dtype=o.dtype, pin_memory=True) for o in outs]
        torch.cuda.synchronize(dev)

        def e2e_step():
            d_ev.copy_(pin_ev, non_blocking=True)
            d_off.copy_(pin_off, non_blocking=True)
            step()
            for o, p in zip(outs, pin_out):
                p.copy_(o.reshape(-1), non_blocking=True)

        e2e_step()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        b.record()
        barrier()
        ms = a.elapsed_time(b)
        ms = max_over_ranks(ms, world, dev)
        assert int(pin_out[-1].numpy().view(argus.STATUS_DTYPE)[0]["code"]) == 0
        e2e = {"value": whole_job_rate(n_events, world, ms / args.e2e_steps), "unit": UNIT,
               "h2d_bytes_per_step": int(pin_ev.numel() + pin_off.numel() * 8),
               "d2h_bytes_per_step": int(sum(p.numel() * p.element_size() for p in pin_out)),
               "steps": args.e2e_steps, "ms_per_step": ms / args.e2e_steps,
               "note": "host events in, tables + overlap + offsets + status out; the interval array stays on the device "
                       f"(copying it back would add {n_events // 2 * 48} bytes per step)"}
        del pin_ev

    # The other numbers the contract asks for, a few steps each (world size 1 only): the plain three-call sequence and
    # a single corrupted marker on the bench workload, and the one-call step on the other trace shapes.
    other = None
    if world == 1 and not args.no_other and not args.three_calls:
        other = []

        def record(run, name, step_name, local, steps):
            ms, _, kms, _ = run.timed(local, steps, 3)
            per = ms / steps
            gbs = ALG_BYTES_PER_EVENT * run.n / (per * 1e-3) / 1e9
            other.append({"workload": name, "step": step_name, "events": run.n, "steps": steps, "ms_per_step": per,
                          "events_per_s": run.n / (per * 1e-3), "pipeline_frac": gbs / peak, "kernel_ms": kms})

        three = Runner(spec, d_ev, d_off)  # its own output buffers
        record(three, spec.name, "argus_pair_intervals + argus_aggregate + argus_overlap (three plain calls)",
               three.step_three_calls, max(args.steps // 2, 3))
        del three
        torch.cuda.empty_cache()
        if spec.name == "decode_megakernel" and not args.iters:
            # one end marker of stream 0 turned into the end of another region: stream 0 loses an interval, every later
            # stream's base moves, and the second pairing pass has to re-write them
            pos = (int(d_off[0].item()) + 5) * 16 + 8
            old = int(d_ev[pos].item())
            assert old == 7  # end of sync_wait (region 3)
            d_ev[pos] = 5    # end of tile_work (region 2)
            try:
                record(main_run, spec.name + " with one corrupted end marker in stream 0", "argus_synthesize",
                       main_run.step_one_call, max(args.steps // 2, 3))
                other[-1]["ambig_required"] = int(state["pair"].fetch_status()["ambig_required"])
            finally:
                d_ev[pos] = old
        for idx in (1, 2, 4):
            if idx == args.workload:
                continue
            sp = tg.config(idx)
            o_ev, o_off = tg.generate_cuda(sp, dev)
            run = Runner(sp, o_ev, o_off)
            record(run, sp.name, "argus_synthesize", run.step_one_call, 10)
            del run, o_ev, o_off
            torch.cuda.empty_cache()

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        oracle.build()
        ev, offs, csm, nsm = oracle_sample(tg, spec, args.cpu_ctas)
        t0 = time.perf_counter()
        oracle_step(oracle, ev, offs, spec, csm, nsm)
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": len(ev) / dt, "unit": UNIT, "cores": 1, "kind": "oracle", "host_cores": os.cpu_count(),
                        "seconds": dt,
                        "sample": f"first {len(csm)} CTAs = {len(offs) - 1} streams, {len(ev)} events, one pass"}
        # the same oracle as independent instances, one CTA of the trace each, on all host cores
        # (the C++ oracle runs outside the interpreter lock; each instance is still single-threaded)
        from concurrent.futures import ThreadPoolExecutor
        ncores = len(os.sched_getaffinity(0))
        offs_all = tg.host_offsets(spec)
        W = spec.warps_per_cta

        nc = min(ncores, spec.num_ctas)
        parts = [(tg.host_streams(spec, offs_all, c * W, (c + 1) * W),
                  (offs_all[c * W:(c + 1) * W + 1] - offs_all[c * W]).astype(np.uint64)) for c in range(nc)]

        def one_cta(part):
            oracle_step(oracle, part[0], part[1], spec, np.zeros(1, np.uint32), 1)
            return len(part[0])

        with ThreadPoolExecutor(ncores) as pool:
            t0 = time.perf_counter()
            done = list(pool.map(one_cta, parts))
            wall = time.perf_counter() - t0
        cpu_baseline["all_cores"] = {"value": sum(done) / wall, "unit": UNIT, "cores": ncores, "seconds": wall,
                                     "sample": f"{nc} CTAs ({sum(done)} events), one single-threaded oracle instance per core"}
        del parts

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64",
            "data": "synthetic",
            "config": {"workload": spec.name, "events_per_gpu": n_events, "streams": S, "regions": spec.num_regions,
                       "input_bytes_per_gpu": n_events * 16, "l2": "inputs (>= 1 GB) are larger than the 126 MB L2",
                       "step": ("argus_pair_intervals + argus_aggregate + argus_overlap" if args.three_calls else
                                "argus_synthesize (pair + aggregate + overlap in one call)") + " on one trace per GPU",
                       "exchange": "kernel-scope tables of all ranks combined by all-reduce every step" if combine else "none"},
            "clocks": sampler.summary(), "e2e": e2e, "gpu_launches": int(launches), "roofline": roofline,
            "cpu_baseline": cpu_baseline, "kernel_ms": kernel_ms, "other": other,
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

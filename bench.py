#!/usr/bin/env python
"""Benchmark of the trace-aggregation hot path.

A step is one pass of the whole path over the 2^30-record trace (benchmark configuration
index 3: 8 chunks of 2^27 records, 4096 apps, 128 ops x 65536 shapes Zipf(1.1)):
reset -> 8 x ingest -> finalize (totals, weights, roofline, compaction) -> top-k per phase.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `value` is records/s with the records resident in HBM;
`e2e` is the same pass through the host-buffer entry point (pinned host -> device copies and
the device -> host read of the result inside the timed region); `roofline` is the ingest
kernel's algorithmic bytes (16 B per record) over its CUDA-event duration against the measured
HBM copy bandwidth; `cpu_baseline` is the CPU oracle timed on this machine on a bounded sample.
`--impl reference` times that oracle alone (there is no other reference implementation).
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

METRIC = "trace records aggregated/sec"
# DRAM bytes (read + written) per 2^27-record ingest call of this workload, from the one-kernel ncu
# captures of the 2^25-record case summarised under profiles/ (traffic grows in proportion to the
# records of a launch, so refresh this constant from the small case, never from a full-size capture):
# scatter_kernel 4 x 0.9895 GB per 2^27-record launch, plus the two drains inside a step's eight calls
# (557 M spilled 12-byte entries at 14.8 B of traffic each -- queued entries and prefetched lines are
# read twice -- and per drain 1.0 GB of table reads and write-backs) spread over the eight calls.
NCU_DRAM_BYTES_PER_INGEST_CALL = 4 * 0.9895e9 + (557e6 * 14.8 + 2 * 1.0e9) / 8
UNIT = "records/s"
WORKLOAD_INDEX = 3
RECORD_BYTES = 16


def measured_peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons every 200 ms while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.gpu_id = gpu_id
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "200"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, smax, power, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); smax.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


def host_threads() -> int:
    return os.cpu_count() or 1


def time_oracle(spec, recs_np, threads: int):
    """Oracle pass over a host sample: reset-free create, ingest, finalize, top-k. Returns seconds."""
    import oracle
    o = oracle.Oracle(spec.app_weights, spec.n_phases)
    o.set_work(spec.work_table())
    t0 = time.perf_counter()
    used = o.ingest(recs_np, threads=threads)
    o.finalize(spec.peak_bw, spec.peak_flops)
    for phase in range(spec.n_phases):
        o.topk(spec.peak_bw, spec.peak_flops, phase, spec.topk)
    dt = time.perf_counter() - t0
    o.close()
    return dt, used


def sample_records(spec, count: int):
    """First `count` records of the workload as a numpy array (GPU sampler when available)."""
    import numpy as np
    import tracegen as tg
    try:
        import torch
        if torch.cuda.is_available():
            from tracegen.gpu import GpuSampler
            out = torch.empty(count * RECORD_BYTES, dtype=torch.uint8, device="cuda:0")
            GpuSampler(spec, "cuda:0").fill(out, 0, count)
            torch.cuda.synchronize()
            return out.cpu().numpy().view(tg.RECORD_DTYPE)
    except Exception:
        pass
    return tg.generate(spec, 0, count)


def run_reference(args):
    """The oracle as it stands, timed on the host cores on a bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from tracegen.configs import make_spec
    spec = make_spec(WORKLOAD_INDEX)
    spec.work_table()
    count = args.ref_records
    recs = sample_records(spec, count)
    threads = host_threads()
    for _ in range(args.warmup):
        time_oracle(spec, recs[: max(count // 16, 1)], threads)
    t0 = time.perf_counter()
    used = threads
    for _ in range(args.steps):
        _, used = time_oracle(spec, recs, threads)
    dt = time.perf_counter() - t0
    value = count * args.steps / dt
    sample = f"first {count} records of the {spec.name} trace per step ({spec.n} in the full workload)"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u64/u128 integer, f64 ratios",
            "data": "synthetic", "config": {"workload": f"config[{WORKLOAD_INDEX}] {spec.name}", "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def run_ours(args):
    import numpy as np
    import torch
    import torch.distributed as dist
    import paper_2607_14541_b200 as p
    from tracegen.configs import make_spec
    from tracegen.gpu import GpuSampler

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=torch.device(f"cuda:{local}"))
    elif args.force_exchange:
        # one GPU, but the step of a multi-GPU run: a process group of one rank (exercises the exchange path)
        if "MASTER_PORT" in os.environ and "RANK" in os.environ:
            # started by torch.distributed.run with one process: its store is the rendezvous (a tcp://
            # address of our own would be taken for the agent's and never answer)
            os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
            dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device(f"cuda:{local}"))
        else:
            import socket
            with socket.socket() as sock:
                sock.bind(("127.0.0.1", 0))
                port = sock.getsockname()[1]
            dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1,
                                    device_id=torch.device(f"cuda:{local}"))
    sharded = world > 1 or args.force_exchange
    torch.cuda.set_device(local)
    dev = torch.device(f"cuda:{local}")

    spec = make_spec(args.workload)      # the default is the configuration the metric is quoted on
    n = args.records or spec.n
    n_chunks = spec.n_chunks
    chunk = n // n_chunks
    n = chunk * n_chunks
    work = spec.work_table()

    # this rank's partition of the trace: records [rank * n, (rank + 1) * n) of the seeded law
    records = torch.empty(n * RECORD_BYTES, dtype=torch.uint8, device=dev)
    sampler = GpuSampler(spec, dev)
    sampler.fill(records, start=rank * n, count=n)
    torch.cuda.synchronize()

    agg = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work), device=local)
    agg.set_work_table(work)
    out = torch.empty(spec.max_keys * 48, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream(dev)
    ingest_events = []
    owner = None
    if sharded:
        # several GPUs: this rank's handle holds its slice of the trace; a second handle holds the keys
        # this rank owns after the exchange step (every entry travels to its key's owner)
        from paper_2607_14541_b200 import distributed as D
        owner = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, max_work_rows=len(work), device=local)
        owner.set_work_table(work)
        out_owner = torch.empty(spec.max_keys * 48, dtype=torch.uint8, device=dev)

    def step(timed: bool):
        agg.reset()
        if owner is not None:
            owner.reset()
        for c in range(n_chunks):
            view = records[c * chunk * RECORD_BYTES: (c + 1) * chunk * RECORD_BYTES]
            if timed:
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                agg.ingest(view, n=chunk)
                e1.record(stream)
                ingest_events.append((e0, e1))
            else:
                agg.ingest(view, n=chunk)
        if owner is not None:
            _, n_out = D.aggregate_sharded(agg, owner, spec.peak_bw, spec.peak_flops, out_local=out, out_owner=out_owner)
            tops = [D.global_topk(owner, phase, spec.topk) for phase in range(spec.n_phases)]
            return n_out, tops
        _, n_out = agg.finalize(spec.peak_bw, spec.peak_flops, out=out)
        tops = [agg.topk(phase, spec.topk) for phase in range(spec.n_phases)]
        return n_out, tops

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        n_keys, tops = step(False)
    barrier()
    sampler_clk = ClockSampler(_gpu_id(torch, local))
    sampler_clk.start()
    launches0 = agg.launch_count()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record(stream)
    for _ in range(args.steps):
        n_keys, tops = step(True)
    ev1.record(stream)
    barrier()
    elapsed_ms = ev0.elapsed_time(ev1)
    launches = agg.launch_count() - launches0 + (owner.launch_count() if owner is not None else 0)
    ingest_ms = [a.elapsed_time(b) for a, b in ingest_events]
    st = agg.stats()
    assert st["n_valid"] + st["n_rejected"] == n and st["n_dropped"] == 0, st

    # end to end: pinned host records -> ingest_host -> finalize -> entries read back to the host
    e2e = None
    if not args.no_e2e:
        e2e = run_e2e(args, torch, p, spec, agg, records, out, n, world, barrier)
    clocks = sampler_clk.stop()

    t = torch.tensor([elapsed_ms, e2e["ms"] if e2e else 0.0], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    elapsed_ms, e2e_ms = float(t[0]), float(t[1])

    if rank == 0:
        value = world * n * args.steps / (elapsed_ms * 1e-3)
        peak, peak_src = measured_peak_hbm()
        mean_ingest_ms = statistics.mean(ingest_ms)
        achieved = chunk * RECORD_BYTES / (mean_ingest_ms * 1e-3) / 1e9
        traffic = args.ncu_traffic_bytes
        if traffic is None and chunk == (1 << 27) and args.workload == WORKLOAD_INDEX:
            traffic = NCU_DRAM_BYTES_PER_INGEST_CALL
        roofline = {"bound": "hbm", "kernel": "ingest pass: scatter_kernel (dominant) + partition_kernel drains",
                    "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                    "algorithmic_bytes_per_launch": chunk * RECORD_BYTES, "launch_ms_mean": mean_ingest_ms,
                    "launch_ms_best": min(ingest_ms), "peak_source": peak_src,
                    "frac_of_nominal_8TBs": achieved / 8000.0,
                    "note": "duration = CUDA events around each ingest call (scatter launch + partition launch, "
                            "which drains the spill buffers when one passes 3/4 of its capacity: calls 4 and 8 "
                            "here); call 0 of a step also holds the "
                            "hot-directory build; achieved = 16 B x records / duration"}
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": elapsed_ms / args.steps, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "u64/u128 integer, f64 ratios", "data": "synthetic",
                "config": {"workload": f"config[{args.workload}] {spec.name}: {n} records/GPU in {n_chunks} chunks, "
                                       f"{spec.n_apps} apps, {spec.n_ops} ops x {spec.n_shapes} shapes Zipf({spec.zipf_s})",
                           "records_per_gpu": n, "chunks": n_chunks, "live_keys": int(n_keys),
                           "l2": "inputs (16 GiB per step) exceed L2; no flush needed",
                           "step": ("reset + ingest x chunks + finalize + topk per phase" if not sharded else
                                    "reset + ingest x chunks + exchange step (entries grouped by key owner, NCCL "
                                    "all-to-all, merge at the owner, totals combined, finalize of the owned keys) "
                                    "+ global topk per phase (owners' candidates gathered and ranked)"),
                           "live_keys_is": "keys of this GPU's trace" if not sharded else "keys rank 0 owns",
                           "workspace_bytes_per_handle": agg.workspace_bytes,
                           "parallelism": f"trace sharded by records x{world}"},
                "clocks": clocks, "gpu_launches": int(launches), "roofline": roofline,
                "algorithmic_GBps_whole_step": world * n * RECORD_BYTES * args.steps / (elapsed_ms * 1e-3) / 1e9}
        if e2e:
            line["e2e"] = {"value": world * e2e["records"] * e2e["steps"] / (e2e_ms * 1e-3), "unit": UNIT,
                           "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"],
                           "steps": e2e["steps"], "sample": e2e["sample"]}
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(args, spec, records, torch)
        if world == 1 and not args.no_per_config and not sharded and args.workload == WORKLOAD_INDEX and n == spec.n:
            del agg
            line["per_config"] = per_config(torch, p, records, n, peak)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
    if sharded:
        dist.destroy_process_group()


# DRAM bytes moved per record by the ingest pass (scatter launches + the drains they trigger), from
# one-kernel ncu captures of 2^25..2^27-record cases summarised under profiles/ (traffic grows in
# proportion to the records of a launch); None where no capture was taken.
NCU_DRAM_BYTES_PER_RECORD = {0: 17.8, 1: 21.5, 2: 46.8, 3: NCU_DRAM_BYTES_PER_INGEST_CALL / float(1 << 27), 4: 19.9}


def per_config(torch, p, records3, n3, peak):
    """The ingest pass of each of the five benchmark configurations, timed the same way: records resident
    in HBM, reset (untimed), CUDA events around all ingest calls of the configuration, best of three after
    a warm-up.  Config 3's records are the bench step's own."""
    from tracegen.configs import make_spec
    from tracegen.gpu import GpuSampler
    rows = []
    # the five configurations, then the tiny configuration's law at 2^28 records: every one of its 4096
    # keys sits in the shared-memory directory, which shows the rate of the path when nothing spills
    for index, n_override in ((0, None), (1, None), (2, None), (3, None), (4, None), (0, 1 << 28)):
        spec = make_spec(index) if n_override is None else make_spec(index, n=n_override)
        if index == WORKLOAD_INDEX:
            recs, n = records3, n3
        else:
            n = spec.n
            recs = torch.empty(n * RECORD_BYTES, dtype=torch.uint8, device=records3.device)
            GpuSampler(spec, records3.device).fill(recs, 0, n)
        chunk = n // spec.n_chunks
        agg = p.Aggregator(spec.app_weights, spec.n_phases, spec.max_keys, device=records3.device.index)
        best = None
        for rep in range(4):
            agg.reset()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for c in range(spec.n_chunks):
                agg.ingest(recs[c * chunk * RECORD_BYTES:(c + 1) * chunk * RECORD_BYTES], n=chunk)
            e1.record()
            torch.cuda.synchronize()
            ms = e0.elapsed_time(e1)
            if rep > 0 and (best is None or ms < best):
                best = ms
        st = agg.stats()
        gbs = chunk * spec.n_chunks * RECORD_BYTES / (best * 1e-3) / 1e9
        rows.append({"config": index, "name": spec.name if n_override is None else f"{spec.name} law, {n_override} records",
                     "records": chunk * spec.n_chunks, "ingest_ms": best,
                     "records_per_s": chunk * spec.n_chunks / (best * 1e-3), "algorithmic_GBps": gbs,
                     "frac_of_measured": gbs / peak, "frac_of_nominal_8TBs": gbs / 8000.0,
                     "spill_fraction": st["n_spilled"] / max(st["n_valid"], 1), "live_keys": st["n_keys"],
                     "drains": int(st["n_drains"]),
                     "dram_bytes_per_record": NCU_DRAM_BYTES_PER_RECORD.get(index),
                     "note": "16 MiB of records: L2-resident and launch-bound, not an HBM measurement"
                             if index == 0 and n_override is None else None})
        del agg
        if index != WORKLOAD_INDEX:
            del recs
        torch.cuda.empty_cache()
    return rows


def _gpu_id(torch, local: int) -> str:
    try:
        return "GPU-" + str(torch.cuda.get_device_properties(local).uuid)
    except Exception:
        return str(local)


def run_e2e(args, torch, p, spec, agg, records, out, n, world, barrier):
    import psutil
    avail = psutil.virtual_memory().available
    n_host = n
    while n_host * RECORD_BYTES * world * 1.5 > avail and n_host > (1 << 22):
        n_host //= 2
    host = torch.empty(n_host * RECORD_BYTES, dtype=torch.uint8, pin_memory=True)
    host.copy_(records[: n_host * RECORD_BYTES])
    host_out = torch.empty(out.numel(), dtype=torch.uint8, pin_memory=True)
    torch.cuda.synchronize()
    steps = max(1, min(args.steps, args.e2e_steps))
    d2h = 0

    def step():
        nonlocal d2h
        agg.reset()
        agg.ingest_host(host, n=n_host)
        _, n_out = agg.finalize(spec.peak_bw, spec.peak_flops, out=out)
        host_out[: n_out * 48].copy_(out[: n_out * 48], non_blocking=True)
        tops = [agg.topk(phase, spec.topk) for phase in range(spec.n_phases)]
        torch.cuda.synchronize()
        d2h = n_out * 48 + sum(len(t) for t in tops) * 48
    step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(steps):
        step()
    barrier()
    ms = (time.perf_counter() - t0) * 1e3
    sample = "full workload" if n_host == n else f"first {n_host} records (host RAM bound)"
    return {"ms": ms, "records": n_host, "steps": steps, "h2d": n_host * RECORD_BYTES, "d2h": d2h, "sample": sample}


def cpu_baseline(args, spec, records, torch):
    import numpy as np
    import tracegen as tg
    count = args.cpu_records
    recs = records[: count * RECORD_BYTES].cpu().numpy().view(tg.RECORD_DTYPE)
    threads = host_threads()
    dt, used = time_oracle(spec, recs, threads)
    single = min(count, 1 << 22)                       # the same oracle on one thread, a shorter prefix
    dt1, _ = time_oracle(spec, recs[:single], 1)
    return {"value": count / dt, "unit": UNIT, "cores": used, "kind": "oracle", "seconds": dt,
            "sample": f"first {count} records of the workload, std::map group-by on {used} threads + finalize + topk",
            "single_thread": {"value": single / dt1, "unit": UNIT, "seconds": dt1,
                              "sample": f"first {single} records, one thread"}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--records", type=int, default=0, help="records per GPU (default: the full 2^30 workload)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true")
    ap.add_argument("--workload", type=int, default=WORKLOAD_INDEX, choices=range(5),
                    help="benchmark configuration to run the step on (default: the one the metric is quoted on; "
                         "the others are for profiling small cases)")
    ap.add_argument("--force-exchange", action="store_true",
                    help="with one GPU: run the step of a multi-GPU run (exchange, merge, global top-k) in a process group of one rank")
    ap.add_argument("--cpu-records", type=int, default=1 << 25)
    ap.add_argument("--ref-records", type=int, default=1 << 24)
    ap.add_argument("--ncu-traffic-bytes", type=float, default=None,
                    help="dram bytes per ingest launch from the committed ncu capture (profiles/)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

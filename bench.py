"""Benchmark: pruned-graph forward + generated backward of f = x*sin(a*x+b), elements/s.

One step = one pass of the whole hot path over one batch: the compiled function that fetches
df/dx (per element), df/da and df/db (summed over all elements) runs once over x fp32[2^26]
(per GPU).  Timed with CUDA events on the launching stream; the input (256 MiB) plus the output
(256 MiB) exceed the L2, so every step streams from HBM.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]
"""
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

from paper_1707_08265_b200 import workloads as wl  # noqa: E402

N_ELEMS = 1 << 26
METRIC = "pruned-graph fwd+bwd elements/sec"
UNIT = "elements/s"
WORKLOAD = "config 2: f=x*sin(a*x+b), x fp32[2^26], fetch df/dx, df/da, df/db"
ALG_BYTES_PER_ELEM = 8.0     # read x once, write df/dx once
# dram__bytes_read.sum + dram__bytes_write.sum of the VM kernel per element, from one ncu capture of this
# kernel binary on this workload at 2^25 elements (traffic is proportional to the element count); None once the
# kernel has changed since the counters were taken
NCU_DRAM_BYTES_PER_ELEM = (134.344448e6 + 89.499136e6) / (1 << 25)


def measured_peak_gbs():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons with NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.samples, self.reasons, self.max_mhz = index, False, [], set(), None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.02)

    def summary(self):
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons)}


def oracle_rate(seconds_budget=12.0):
    """The CPU oracle, as it stands, on a bounded sample of the same workload."""
    from oracle import interp
    n = 1 << 21
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, wl.BASE_SEED + 2)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outs = [ids["dx"], ids["da"], ids["db"]]
    interp.run_function(g.desc, inputs, outs, [x, a, b])
    reps, t0 = 0, time.perf_counter()
    while True:
        interp.run_function(g.desc, inputs, outs, [x, a, b])
        reps += 1
        if time.perf_counter() - t0 > seconds_budget or reps >= 64:
            break
    dt = time.perf_counter() - t0
    return reps * n / dt, "%d passes of the fp64 NumPy interpreter over x[2^21] (same graph, same fetches)" % reps, dt / reps


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    per = []
    for _ in range(args.warmup):
        oracle_rate(0.5)
    t0 = time.perf_counter()
    sample = ""
    for _ in range(args.steps):
        rate, sample, _ = oracle_rate(max(1.0, 60.0 / max(1, args.steps)))
        per.append(rate)
    dt = time.perf_counter() - t0
    value = float(np.mean(per))
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * dt / max(1, args.steps), "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "note": "each step is a bounded sample: " + sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def run_other_config(args):
    """Device-resident timing of the other workloads (same step definition: one dragon_run)."""
    import torch
    from paper_1707_08265_b200 import binding as B
    seeds = json.load(open(os.path.join(ROOT, "tests", "golden", "config_seeds.json")))
    tdt = {"f32": torch.float32, "bf16": torch.bfloat16, "i32": torch.int32}
    gen = torch.Generator("cuda").manual_seed(wl.BASE_SEED + args.config)

    def dev_random(g, t):
        ti = g.desc["tensors"][t]
        if ti["dtype"] == "i32":
            return torch.randint(0, 4096, tuple(ti["shape"]), generator=gen, device="cuda", dtype=torch.int32)
        return torch.empty(tuple(ti["shape"]), dtype=torch.float32, device="cuda").normal_(generator=gen).to(tdt[ti["dtype"]])

    if args.config == 1:
        n = 1 << 20
        g, ids = wl.toy_function(n)
        inputs, outputs, units, what = [ids["x"], ids["a"], ids["b"]], [ids["f"], ids["y"]], n, "f and y of x*sin(a*x+b), x fp32[2^20] (L2-resident)"
    elif args.config == 3:
        n = 1 << 27
        g, inputs, outputs = wl.random_dag(n, seeds["random_dag"]["seed"])
        units, what = n, "random 64-operator elementwise DAG, 4 x fp32[2^27], 2 fetches"
    elif args.config == 6:   # not one of the five: the SGD weight update as a graph of its own, 12 bytes per element
        n = 1 << 26
        g, ids = wl.updater([n], "sgd")
        inputs, outputs, units, what = [ids["W"], ids["g"], ids["lr"]], [ids["W_new"]], n, "SGD updater W - lr*g, fp32[2^26] (memory-bound: 12 B/element)"
    elif args.config == 4:
        g, ids = wl.mlp(8192, 4096, 4096, 4096)
        inputs = [ids[k] for k in ("X", "W1", "b1", "W2", "b2", "labels")]
        outputs = [ids[k] for k in ("loss", "dW1", "db1", "dW2", "db2")]
        units, what = 8192, "MLP 8192 x 4096-4096-4096 bf16, forward + backward (batch rows per step)"
    else:
        from oracle import prune as oprune   # which inputs are connected is decided outside the generator
        g, inputs, fetch = wl.random_row_dag(16384, 4096, seeds["random_row_dag"]["seed"])
        if args.config == 5:
            G = oprune.backward_marks(g.desc, fetch, inputs)
            outputs = fetch + g.grad(fetch, [i for i in inputs if i in G])
            units, what = 16384 * 4096, "random 1024-operator row DAG on [16384,4096], forward + backward"
        else:   # not one of the five: the same DAG with one gradient stage per objective (Jacobian-style fetches)
            outputs = list(fetch)
            for o in fetch:
                G = oprune.backward_marks(g.desc, [o], inputs)
                outputs += g.grad([o], [i for i in inputs if i in G])
            units, what = 16384 * 4096, "row DAG on [16384,4096], forward + one gradient stage per objective (%d fetches)" % len(outputs)
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    feeds = [dev_random(g, t) if u else None for t, u in zip(inputs, f.used_inputs())]
    if args.config == 4:
        for j in (1, 2, 3, 4):
            feeds[j] = (feeds[j].float() / 64).to(torch.bfloat16)
    outs = [torch.empty(tuple(g.shape(t)), dtype=tdt[g.desc["tensors"][t]["dtype"]], device="cuda") for t in outputs]
    for _ in range(max(3, args.warmup)):
        f.run_torch(feeds, outs)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    steps = min(args.steps, 50)
    e0.record()
    for _ in range(steps):
        f.run_torch(feeds, outs)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    assert f.status() == 0
    nbytes = sum(t.numel() * t.element_size() for t in feeds if t is not None) + sum(t.numel() * t.element_size() for t in outs)
    line = {"config": args.config, "workload": what, "ms_per_step": ms, "units_per_s": units / (ms * 1e-3),
            "io_GBps": nbytes / ms / 1e6, "launches": f.num_launches(), "plan": f.describe().strip().split("\n")[:24]}
    if args.config == 4:
        line["gemm_TFLOPs_over_whole_step"] = 5 * 2 * 8192 * 4096 * 4096 / ms / 1e9
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--elements", type=int, default=N_ELEMS, help="elements per GPU (default: the benchmark's 2^26)")
    ap.add_argument("--skip-cpu-baseline", action="store_true")
    ap.add_argument("--config", type=int, default=2, choices=[1, 2, 3, 4, 5, 6, 7],
                    help="2 (default) is the benchmark workload; the others print one summary line each (6: SGD updater)")
    args = ap.parse_args()
    if args.impl == "reference":
        return run_reference(args)
    if args.config != 2:
        return run_other_config(args)

    import torch
    import torch.distributed as dist
    from paper_1707_08265_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    n = args.elements
    warm = max(3, args.warmup)

    # every rank owns its own shard of x (weak scaling); a and b are shared scalars
    g, ids = wl.toy_function_grad(n)
    x, a, b = wl.toy_feeds(n, wl.BASE_SEED + 2 + 1000 * rank)
    _, a, b = wl.toy_feeds(4, wl.BASE_SEED + 2)
    inputs = [ids["x"], ids["a"], ids["b"]]
    outputs = [ids["dx"], ids["da"], ids["db"]]
    f = B.Graph.from_desc(g.desc).function(inputs, outputs)
    f.ensure_workspace()
    stream = torch.cuda.Stream()
    d_feeds = [torch.from_numpy(np.ascontiguousarray(v)).cuda() for v in (x, a, b)]
    d_out = [torch.empty(tuple(g.shape(o)), dtype=torch.float32, device="cuda") for o in outputs]
    feed_ptrs = [t.data_ptr() for t in d_feeds]
    fetch_ptrs = [t.data_ptr() for t in d_out]

    from paper_1707_08265_b200 import sharding

    def evaluate():
        f.run(feed_ptrs, fetch_ptrs, stream.cuda_stream)
        return d_out

    def step():
        if world == 1:
            evaluate()
        else:  # the one exchange of the sharded path: the two summed gradients
            with torch.cuda.stream(stream):
                sharding.run_sharded(evaluate, [1, 2], lambda t: dist.all_reduce(t))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(warm):
        step()
    barrier()
    vm_step = 0   # the plan of this function is one VM step (plus its finishing reduction)
    f.profile(vm_step, args.steps)
    sampler = ClockSampler(local)
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for _ in range(args.steps):
        step()
    e1.record(stream)
    barrier()
    sampler.stop_flag = True
    ms = e0.elapsed_time(e1)
    kern_ms, kern_runs = f.profile_read()
    f.profile(-1, 0)
    if world > 1:
        t = torch.tensor([ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ms = float(t.item())
    value = world * n * args.steps / (ms * 1e-3)

    # end to end: the same step through the host-buffer entry point, copies inside the timed region
    h_x = torch.from_numpy(np.ascontiguousarray(x)).pin_memory()
    h_a, h_b = torch.from_numpy(np.ascontiguousarray(a)).pin_memory(), torch.from_numpy(np.ascontiguousarray(b)).pin_memory()
    h_out = [torch.empty(tuple(g.shape(o)), dtype=torch.float32).pin_memory() for o in outputs]
    stg_bytes = f.staging_bytes()
    stg = torch.empty(stg_bytes + 256, dtype=torch.uint8, device="cuda")
    stg_ptr = (stg.data_ptr() + 255) & ~255
    hf = [h_x.data_ptr(), h_a.data_ptr(), h_b.data_ptr()]
    ho = [t.data_ptr() for t in h_out]
    e2e_steps = max(3, min(args.steps, 20))
    for _ in range(2):
        f.run_host(hf, ho, stg_ptr, stg_bytes, stream.cuda_stream)
    barrier()
    e0.record(stream)
    for _ in range(e2e_steps):
        f.run_host(hf, ho, stg_ptr, stg_bytes, stream.cuda_stream)
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1)
    if world > 1:
        t = torch.tensor([e2e_ms], dtype=torch.float64, device="cuda")
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        e2e_ms = float(t.item())
    assert f.status() == 0
    # the host copies came back: a cheap end-to-end sanity check against the device-resident run
    assert np.array_equal(h_out[0][:1024].numpy(), d_out[0][:1024].cpu().numpy())

    if rank == 0:
        peak, peak_kind = measured_peak_gbs()
        kern_avg_ms = kern_ms / max(1, kern_runs)
        achieved = ALG_BYTES_PER_ELEM * n / (kern_avg_ms * 1e-3) / 1e9
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warm,
                "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": WORKLOAD, "elements_per_gpu": n, "l2": "inputs+outputs (512 MiB) larger than L2",
                           "plan": f.describe().strip().split("\n")},
                "clocks": sampler.summary(),
                "e2e": {"value": world * n * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
                        "h2d_bytes_per_step": 4 * n + 8, "d2h_bytes_per_step": 4 * n + 8},
                "gpu_launches": f.num_launches() * args.steps,
                "roofline": {"bound": "hbm", "kernel": "dragon_vm_dense", "achieved": achieved, "peak": peak, "unit": "GB/s",
                             "frac": achieved / peak, "peak_kind": "of " + peak_kind, "traffic": None if NCU_DRAM_BYTES_PER_ELEM is None else NCU_DRAM_BYTES_PER_ELEM * n,
                             "kernel_ms": kern_avg_ms, "frac_of_nominal_8TBs": achieved / 8000.0}}
        if not args.skip_cpu_baseline and world == 1:
            rate, sample, _ = oracle_rate()
            line["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the mixed-bit quantized AdamW step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg5] [--impl ours|reference]

One "step" is one pass of the whole hot path over the workload: the fused step kernel over every
tensor, and on decision steps (every K_dec steps of the workload) the fused statistics, their
fetch, and the host transition decision.  Each rank runs an independent replica (the path does not
shard); the line reports the aggregate over ranks.  Rank 0 prints ONE JSON line.
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

from paper_2604_06836_b200 import workloads as W  # noqa: E402

METRIC = "quantized_adamw_step_params_per_s"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per parameter of the step kernel from the ncu captures
# summarised in profiles/ (cfg5s is the cfg5 recipe on 6 layers), scaled by the parameters per launch.
NCU_TRAFFIC_BYTES_PER_PARAM = {"cfg5": 12.376, "cfg5s": 12.376, "cfg2": 14.237}


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period=0.02):
        super().__init__(daemon=True)
        self.period, self.index = period, index
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = torch.cuda.get_device_properties(index).uuid
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
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
        while not self._stop_evt.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        return {"sm_mhz": (float(np.median(self.samples)) if self.samples else None),
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------------
# the oracle arm (CPU baseline / --impl reference)
# ------------------------------------------------------------------------------------------------
FULL_ORACLE_PARAMS = 1 << 27     # workloads up to this size get a full oracle step on their real tensors


def _to_np(t: torch.Tensor) -> np.ndarray:
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.contiguous().view(torch.int16).numpy().view(np.uint16).copy()
    return t.contiguous().numpy().copy()


def oracle_run(w: W.Workload, bits_m, bits_v, budget_s: float, repeats: int = 1):
    """Times the CPU oracle, as it stands, on the machine's host cores.

    Workloads of up to 2^27 parameters (cfg1-cfg3): one full oracle step over the workload's real tensors
    (the seeded parameter and gradient draws of the workload, every tensor at its width), all cores, and the
    same full step again on one thread.  Larger workloads (cfg4, cfg5): a bounded sample, i.e. block-aligned
    chunks of at most 2^18 elements of tensors drawn in proportion to their size (so the sample has the
    workload's numel-weighted width mix), sized for about `budget_s` seconds of all-core work, and a
    single-thread timing on every k-th chunk of the same sample.  Work is spread over host threads
    range by range; the oracle's C code runs outside the interpreter lock."""
    import oracle as O
    from concurrent.futures import ThreadPoolExecutor

    cores = os.cpu_count() or 1
    chunk = 1 << 18
    block = w.block
    kw = dict(lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay,
              v_mode=O.LOG_PL if w.v_log == "pl" else O.LOG)
    if w.grad_dtype == "fp16":
        kw.update(fp16_grad=True, inv_grad_scale=1.0 / w.loss_scale if w.loss_scale > 0 else 1.0)
    full = w.total_params <= FULL_ORACLE_PARAMS
    if full and w.total_params < 4 * cores * chunk:        # a small workload still gets a few ranges per thread
        chunk = max(1024, w.total_params // (4 * cores) // 1024 * 1024)
    numels = w.numels
    rng = np.random.default_rng(0)
    tensors = {}        # tensor index -> [theta, grad, state in, state out]

    def materialise(l: int, n: int, real: bool):
        if real:
            th, g = _to_np(W.draw_param(w, l, "cpu")), _to_np(W.draw_grad(w, l, 1, "cpu"))
        else:   # a chunk-sized stand-in with the value distributions of the recipe (the timing does not depend on values)
            th = rng.normal(0, 0.02, n).astype(np.float32)
            g32 = torch.from_numpy((rng.standard_t(3, n) * 1e-3).astype(np.float32))
            g = _to_np(g32.to({"fp32": torch.float32, "bf16": torch.bfloat16, "fp16": torch.float16}[w.grad_dtype]))
        bm, bv = int(bits_m[l]), int(bits_v[l])
        return [th, g, O.new_state(n, block, bm, bv), O.new_state(n, block, bm, bv)]

    tasks = []          # (key, e0, e1)
    if full:
        for l, n in enumerate(numels):
            tensors[l] = materialise(l, n, True)
            tasks += [(l, e0, min(n, e0 + chunk)) for e0 in range(0, n, chunk)]
        taken = w.total_params
    else:
        st = O.new_state(chunk, block, 4, 4)
        t0 = time.perf_counter()
        O.step(rng.normal(0, 0.02, chunk).astype(np.float32), (rng.standard_t(3, chunk) * 1e-3).astype(np.float32),
               st, block, t=1, lr=w.lr, beta1=w.beta1, beta2=w.beta2, eps=w.eps, weight_decay=w.weight_decay)
        rate1 = chunk / (time.perf_counter() - t0)        # calibration only: sizes the sample
        want = int(min(FULL_ORACLE_PARAMS, max(chunk, rate1 * cores * budget_s)))
        prob = np.asarray(numels, dtype=np.float64) / float(sum(numels))
        taken, k = 0, 0
        while taken < want:
            l = int(rng.choice(len(numels), p=prob))
            n = int(min(chunk, numels[l]))
            n = n // block * block if n >= block else n
            tensors[("s", k)] = materialise(l, n, False)
            tasks.append((("s", k), 0, n))
            taken += n
            k += 1

    def run(task, t):
        key, e0, e1 = task
        th, g, a, b = tensors[key]
        O.step_range(th, g, e0, e1, block, a, b, t=t, **kw)

    def swap():
        for v in tensors.values():
            v[2], v[3] = v[3], v[2]

    times = []
    with ThreadPoolExecutor(max_workers=cores) as ex:
        list(ex.map(lambda tk: run(tk, 1), tasks))          # step 1 populates the states (untimed)
        swap()
        for r in range(repeats):
            t0 = time.perf_counter()
            list(ex.map(lambda tk: run(tk, 2 + r), tasks))
            times.append(time.perf_counter() - t0)
            swap()
    # one thread, same width mix: the whole step for the small workloads, every k-th chunk of the sample otherwise
    sub = tasks if full else tasks[::max(1, len(tasks) // 16)]
    n_sub = sum(e1 - e0 for _, e0, e1 in sub)
    t0 = time.perf_counter()
    for tk in sub:
        run(tk, 2 + repeats)
    single = n_sub / (time.perf_counter() - t0)
    used = min(cores, len(tasks))
    what = (f"one full oracle step over the workload's {len(numels)} real tensors ({taken} params, ranges of <= {chunk} "
            f"elements over {used} threads)" if full else
            f"{taken} params in {len(tasks)} block-aligned chunks of <= {chunk} elements of tensors drawn in proportion "
            f"to their size at their widths, one oracle step each, {used} threads")
    return {"params": taken, "seconds": times, "cores": used, "single_thread": single,
            "single_thread_sample": f"{n_sub} params ({len(sub)} of the same chunks), 1 thread", "sample": what,
            "host_cores": cores}


def run_reference(args, w, bits_m, bits_v):
    rank, _, world = dist_env()
    if rank != 0:
        return
    res = oracle_run(w, bits_m, bits_v, budget_s=max(2.0, 60.0 / max(1, args.steps + args.warmup)),
                     repeats=args.steps + args.warmup)
    timed = res["seconds"][args.warmup:]
    sec = float(np.mean(timed))
    value = res["params"] / sec
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "params": w.total_params, "block": w.block, "grad_dtype": w.grad_dtype,
                   "mean_bits": W.mean_bits(w, bits_m, bits_v),
                   "step_is": ("one full oracle step over the workload" if w.total_params <= FULL_ORACLE_PARAMS
                               else "one oracle step over the bounded sample")},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": res["cores"], "kind": "oracle", "sample": res["sample"],
                         "host_cores": res["host_cores"], "single_thread_value": res["single_thread"],
                         "single_thread_sample": res["single_thread_sample"]},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------
def run_ours(args, w, bits_m, bits_v):
    from paper_2604_06836_b200 import stq
    from paper_2604_06836_b200.runner import Job

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if use_dist:
            dist.barrier()
        torch.cuda.synchronize()

    # --shard: strong scaling.  Every rank keeps the optimizer state of a block-aligned slice of the
    # parameter list and steps only that; the per-layer sums are added over ranks on decision steps.
    w_global, L_global, layer_of_row = w, len(w.shapes), None
    if args.shard:
        from dataclasses import replace
        from paper_2604_06836_b200 import multi as _multi
        mine = _multi.partition(w.numels, world)[rank]
        layer_of_row = np.array([l for l, _, _ in mine], dtype=np.int64)
        w = replace(w, name=w.name + f"-shard{rank}of{world}",
                    shapes=tuple((f"{w.shapes[l][0]}[{lo}:{hi}]", (hi - lo,)) for l, lo, hi in mine))
        bits_m, bits_v = bits_m[layer_of_row], bits_v[layer_of_row]

    layout = args.layout
    if layout == "tile" and w.v_log == "ts" and any(n % w.block for n in w.numels):
        layout = "exact"       # zero padding inside a last, partly real block would change the minimum the two-scale code keeps
    job = Job(w, bits_m, bits_v, device=dev, tile_padded=(layout == "tile"))
    job.draw_grads(1)

    def decide(t):
        st = job.layer_stats()
        if layer_of_row is not None:
            from paper_2604_06836_b200 import multi as _multi
            full = np.zeros((L_global, 4))
            np.add.at(full, layer_of_row, st)
            st = _multi.sync_layer_stats(full, dev)
        pol.decide(st, t)                            # the paper's policy in shadow: widths stay the seeded ones
    pol = stq.Policy(alpha=0.1, tau=100.0, eps_stat=1e-8, interval=w.decision_interval)
    stream = torch.cuda.current_stream()

    def one_step_is_decision(t):
        return t % w.decision_interval == 0         # the t < 5 clause belongs to the start of training

    def one_step(t):
        dec = one_step_is_decision(t)
        job.step(t, stats=dec)
        if dec:
            decide(t)
        return dec

    t = 0
    for k in range(args.warmup):
        t += 1
        if k == args.warmup - 1 and not one_step_is_decision(t):
            # the last warm-up step takes the decision path whatever its index, so that every kernel
            # variant the timed region launches has been loaded before the clock starts
            job.step(t, stats=True)
            decide(t)
        else:
            one_step(t)
    barrier()

    # Timing hygiene: the inputs of a step must not sit in L2 from the step before.  The large
    # configurations touch gigabytes per step; a small one (cfg1: 16 MB) gets an L2 flush (a 256 MB
    # write) before every timed step, and its job time is then the sum of the per-step device times.
    small = job.algorithmic_bytes() < (256 << 20)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev) if small else None

    sampler = ClockSampler(local_rank)
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    is_dec = []
    launches0 = job.handle.launch_count
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record(stream)
    for i in range(args.steps):
        t += 1
        dec = t % w.decision_interval == 0
        if flush is not None:
            flush.zero_()
        ev[i][0].record(stream)
        job.step(t, stats=dec)
        ev[i][1].record(stream)
        if dec:
            decide(t)
        is_dec.append(dec)
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = job.handle.launch_count - launches0
    total_ms = e0.elapsed_time(e1)
    kern_ms = np.array([a.elapsed_time(b) for a, b in ev])
    is_dec = np.array(is_dec)
    if small:
        total_ms = float(kern_ms.sum())

    # ---- cost of the decision step in the paper's order (statistics before the update) ------------------
    # Outside the timed region: the gradient-only pass, the fetch of the per-layer sums and the host
    # decision, i.e. what Algorithm 1 adds every U steps (its O(N/K) overhead); the timed steps use the
    # fused order, whose extra cost is kernel_ms_with_stats - kernel_ms_plain plus the same fetch.
    tbl = job.table()
    job.handle.grad_stats(tbl, job.grad_dtype)
    job.layer_stats()
    g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g0.record(stream)
    for _ in range(5):
        job.handle.grad_stats(tbl, job.grad_dtype)
    g1.record(stream)
    torch.cuda.synchronize()
    grad_stats_ms = g0.elapsed_time(g1) / 5
    h0 = time.perf_counter()
    st_ = job.layer_stats()
    h1 = time.perf_counter()
    pol.decide(st_, t + 1)
    h2 = time.perf_counter()
    job._tbl = None
    decision = {"grad_stats_pass_ms": grad_stats_ms, "stats_fetch_ms": (h1 - h0) * 1e3,
                "host_decide_ms": (h2 - h1) * 1e3, "tensors": job.L}

    # ---- end to end through the host-buffer entry point ----------------------------------------------
    # (the host-buffer entry point and the oracle sample cover the plain step; the fp16 workloads with a
    # loss scale are device-path measurements only)
    amp = w.loss_scale > 0
    e2e = None
    e2e_error = None
    if not args.no_e2e and not amp:
        try:
            e2e = run_e2e(job, w, args)
        except (RuntimeError, MemoryError) as exc:     # e.g. the host cannot pin another 20 GB for this rank
            e2e_error = f"{type(exc).__name__}: {exc}"[:300]

    from paper_2604_06836_b200 import multi
    params = w.total_params
    total_ms, e2e_ms = multi.max_over_ranks([total_ms, e2e["ms"] if e2e else 0.0], dev)   # slowest rank
    job_params = w_global.total_params if args.shard else world * params     # what all ranks process per step
    value = job_params * args.steps / (total_ms * 1e-3)
    alg_bytes = job.algorithmic_bytes()
    k_ms = float(kern_ms.mean())
    achieved = alg_bytes / (k_ms * 1e-3) / 1e9
    peak, peak_kind = measured_peak()
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "strong" if args.shard else "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w_global.name, "params": job_params if args.shard else params, "tensors": len(w.shapes), "block": w.block,
                   "grad_dtype": w.grad_dtype, "loss_scale": w.loss_scale or None, "lp_copy": w.lp_copy or None, "v_log": w.v_log,
                   "mean_bits": round(W.mean_bits(w, bits_m, bits_v), 3),
                   "decision_interval": w.decision_interval, "decision_steps_timed": int(is_dec.sum()),
                   "l2": ("flushed before every timed step (256 MB write; %.1f MB touched per step)" % (alg_bytes / 1e6)
                          if small else "inputs larger than L2 (%.1f GB touched per step)" % (alg_bytes / 1e9)),
                   "parallelism": ("sharded over %d ranks (this rank: %d parameters)" % (world, params) if args.shard
                                   else "replicas" if world > 1 else "single"), "grid": job.handle.grid_size,
                   "layout": ("tile: every tensor's storage padded with zeros to whole 4096-element tiles, padded lengths "
                              "given to the library; parameters and bytes count the real elements only"
                              if layout == "tile" else "exact: tensors at their true lengths"),
                   "state_bytes": job.state_bytes(), "fp32_state_bytes": 8 * params,
                   "state_saved_frac": 1.0 - job.state_bytes() / (8.0 * params)},
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": (NCU_TRAFFIC_BYTES_PER_PARAM[args.config] * params
                                 if args.config in NCU_TRAFFIC_BYTES_PER_PARAM else None),
                     "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": alg_bytes,
                     "bytes_per_param": alg_bytes / params, "kernel_ms_mean": k_ms,
                     "kernel_ms_plain": float(kern_ms[~is_dec].mean()) if (~is_dec).any() else None,
                     "kernel_ms_with_stats": float(kern_ms[is_dec].mean()) if is_dec.any() else None,
                     # the step runs at the board's power limit: the first steps see boost clocks, later ones do not
                     "kernel_ms_first_10": float(kern_ms[:10].mean()), "kernel_ms_last_10": float(kern_ms[-10:].mean()),
                     "frac_of_nominal_8000": achieved / 8000.0},
        "clocks": clocks,
        "decision_step": decision,
        "gpu_launches": int(launches),
        "gpu_params_per_s_per_gpu": params * args.steps / (total_ms * 1e-3),
    }
    if e2e_error:
        line["e2e"] = {"value": None, "unit": UNIT, "h2d_bytes_per_step": None, "d2h_bytes_per_step": None,
                       "error": e2e_error}
    if e2e:
        line["e2e"] = {"value": job_params * e2e["steps"] / (e2e_ms * 1e-3), "unit": UNIT,
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"], "steps": e2e["steps"],
                       "ms_per_step": e2e_ms / e2e["steps"]}
    # ---- the same workload with the other codes of the second moment (device time only, 20 steps each) ---------
    # Extras, not the headline: the default line above is the polynomial log code of the specification.
    if rank == 0 and world == 1 and w.v_log == "poly" and not args.no_variants and not args.shard:
        from dataclasses import replace
        del job
        line["variants"] = {}
        for code in ("pl", "sr", "ts"):
            try:
                torch.cuda.empty_cache()
                wv = replace(w, v_log=code)
                jv = Job(wv, bits_m, bits_v, device=dev)
                jv.draw_grads(1)
                for tt in (1, 2, 3):
                    jv.step(tt)
                v0, v1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                v0.record(stream)
                for tt in range(4, 24):
                    jv.step(tt)
                v1.record(stream)
                torch.cuda.synchronize()
                vms = v0.elapsed_time(v1) / 20
                line["variants"]["v_log=" + code] = {
                    "ms_per_step": vms, "value": params / (vms * 1e-3), "unit": UNIT, "steps": 20,
                    "frac": jv.algorithmic_bytes() / (vms * 1e-3) / 1e9 / peak,
                    "note": "plain steps, no decision steps, first 20 after warm-up"}
                del jv
            except Exception as exc:          # an extra must never cost the line
                line["variants"]["v_log=" + code] = {"error": f"{type(exc).__name__}: {exc}"[:200]}
    if rank == 0 and not args.no_cpu_baseline and world == 1:
        res = oracle_run(w, bits_m, bits_v, budget_s=8.0, repeats=1)
        line["cpu_baseline"] = {"value": res["params"] / res["seconds"][0], "unit": UNIT, "cores": res["cores"],
                                "kind": "oracle", "sample": res["sample"], "host_cores": res["host_cores"],
                                "single_thread_value": res["single_thread"],
                                "single_thread_sample": res["single_thread_sample"]}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if use_dist:
        dist.destroy_process_group()


def run_e2e(job, w, args):
    """The same step through stq_step_host: pinned host buffers in, host buffers out, copies timed."""
    from paper_2604_06836_b200 import stq
    steps = max(1, min(args.e2e_steps, args.steps))
    # the caller's side of the host path: every kind of buffer in one flat pinned allocation
    tbl, host_states, host_p, host_g = job.host_table(flat=True)
    hp = job.hp(job.t + 1)
    job.handle.step_host(tbl, **hp)          # warm-up: grows the device arena
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    h2d = d2h = 0
    for k in range(steps):
        hp = job.hp(job.t + 2 + k)
        h2d, d2h = job.handle.step_host(tbl, **hp)
    torch.cuda.synchronize()
    ms = (time.perf_counter() - t0) * 1e3
    job._tbl = None
    return {"ms": ms, "steps": steps, "h2d": h2d, "d2h": d2h}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", default="cfg5", help="cfg1..cfg5 (default: the 1.5B bandwidth run); gpt2_medium, roberta_large, vit_b32: "
                         "Table 1's other models under fp16 training (device path only)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-variants", action="store_true", help="skip the extra runs with the other codes of the second moment")
    ap.add_argument("--v-log", default="poly", choices=["poly", "pl", "sr", "ts"],
                    help="code of the second moment (default: the polynomial logarithm)")
    ap.add_argument("--layout", default="tile", choices=["exact", "tile"],
                    help="tile (default): every tensor's storage padded with zeros to whole 4096-element tiles, a step is "
                         "one launch; exact: tensors at their true lengths (ragged last tiles take one more launch per step). "
                         "The results on the real elements are the same (tested against the oracle at full size)")
    ap.add_argument("--shard", action="store_true",
                    help="strong scaling: each rank owns a block-aligned slice of the parameter list "
                         "(default: every rank steps a full replica)")
    args = ap.parse_args()
    w = W.config(args.config)
    if args.v_log != "poly":
        from dataclasses import replace
        w = replace(w, name=w.name + "-v" + args.v_log, v_log=args.v_log)
    bits_m, bits_v, _ = W.draw_bits(w)
    if args.impl == "reference":
        run_reference(args, w, bits_m, bits_v)
    else:
        run_ours(args, w, bits_m, bits_v)


if __name__ == "__main__":
    main()

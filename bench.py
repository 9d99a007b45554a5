#!/usr/bin/env python
"""Benchmark of the sync step (+ FedAvg every H-th step) on synthetic buffers.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

A step is one fls_sync_step over all G groups, followed by fls_fedavg when the step counter is a
multiple of H (one fused call on those steps).  Metric: synced params/s = G*P*K / time (logical
parameters, whole job).  Prints one JSON line on rank 0.  The default workload is the largest one that
fits a single GPU, the Llama-3.2-1B-sized FL+HSDP configuration; the 8B-block and GPT-2-small-sized
workloads are timed afterwards and reported under "other_workloads" of the same line.
With N > 1 every rank runs an independent replica of the workload (the path has no inter-GPU exchange);
the time is the maximum over ranks.  Started without a launcher, `--gpus N` starts the N ranks itself.
`--impl reference` times the CPU oracle on a bounded sample of the same workload instead.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import synthetic as sy

METRIC = "synced_params_per_s"
UNIT = "params/s"
DEFAULT_CONFIG = "llama32_1b_fl_hsdp"
OTHER_WORKLOADS = ("llama31_8b_block_fl_fsdp", "gpt2_small_fl_fsdp")
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per group-element and launch, measured with ncu on
# slices of the workloads (one kernel per capture, a few GB on the device); the traffic of these streams grows
# in proportion to the element count, so a launch over N elements moves N times the figure.  Keyed by kernel
# and, for the kernels that read the gradients, by the gradient bytes per element K*e_g.
NCU_TRAFFIC_BYTES_PER_ELEM = {("reduce", 16): 19.46, ("adamw", None): 28.85, ("adamw_fedavg", None): 29.39, ("fedavg", None): 9.54,
                              ("step_noclip", 16): 40.66,
                              # resident step on the tiny workload (captured whole): all reads, and none of the 14 bytes
                              # written per element, which are still in L2 when a kernel over 68 MB ends
                              ("step_resident", 8): 20.03}
# The CPU oracle is timed on the first ORACLE_SAMPLE parameters of every buffer: once on one thread, once with
# the sample cut into chunks that a pool of all host cores works through.
ORACLE_SAMPLE_ONE_CORE = 1 << 24
ORACLE_SAMPLE_ALL_CORES = 1 << 26


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


# --------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples the SM clock and the throttle reasons of one GPU while the timed region runs: the main thread
    reads NVML about once a millisecond while it waits for the region's end event (the region of a small
    workload lasts only tens of ms, too short for nvidia-smi's loop mode).  Falls back to one nvidia-smi
    query if the NVML binding is missing.  Nothing is ever set, only read."""
    REASONS = (("hw_slowdown", 0x8), ("hw_thermal_slowdown", 0x40), ("sw_thermal_slowdown", 0x20), ("sw_power_cap", 0x4),
               ("hw_power_brake_slowdown", 0x80))

    def __init__(self, index: int):
        self.index, self.sm, self.reason_bits, self.power = index, [], 0, []
        self.max_sm, self._nvml = None, None

    def start(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
            self.max_sm = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None

    def _physical_index(self) -> int:
        vis = os.environ.get("CUDA_VISIBLE_DEVICES", "")
        ids = [v for v in vis.split(",") if v.strip() != ""]
        if ids and all(v.strip().isdigit() for v in ids) and self.index < len(ids):
            return int(ids[self.index])
        return self.index

    def sample(self):
        """One reading; called from the main thread while it waits for the timed region's end event."""
        nv = self._nvml
        if nv is None:
            return
        try:
            self.sm.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
            self.reason_bits |= int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)) if hasattr(nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                else int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            self.power.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
        except Exception:
            pass

    def wait_for(self, event):
        """Waits for a CUDA event, sampling the clocks every millisecond or so meanwhile."""
        self.sample()                      # at least one reading, taken while the region is (still) running
        while not event.query():
            time.sleep(0.001)
            self.sample()

    def stop(self) -> dict:
        if self._nvml is None:
            return self._smi_once()
        reasons = [name for name, bit in self.REASONS if self.reason_bits & bit]
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.max_sm, "reasons": reasons,
                "samples": len(self.sm), "power_w_max": max(self.power) if self.power else None, "source": "nvml"}

    def _smi_once(self) -> dict:
        try:
            out = subprocess.run(["nvidia-smi", f"--id={self.index}", "--query-gpu=clocks.sm,clocks.max.sm", "--format=csv,noheader,nounits"],
                                 capture_output=True, text=True, timeout=10).stdout.strip().split(",")
            return {"sm_mhz": float(out[0]), "sm_max_mhz": float(out[1]), "reasons": [], "samples": 1, "source": "nvidia-smi after the region"}
        except Exception:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["clock query unavailable"], "samples": 0}


def max_over_ranks(value: float, world: int, device=None) -> float:
    """Largest `value` over all ranks of the default process group (the job's time is its slowest rank's)."""
    if world <= 1:
        return value
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# --------------------------------------------------------------------------------------- CPU oracle leg
def host_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


def oracle_sample(cfg: dict, sample_params: int, threads: int = 1):
    """One oracle step of all G groups and one FedAvg on the first `sample_params` parameters of every
    buffer, with the oracle's functions as they stand.  threads = 1: the plain whole-array calls on one host
    thread.  threads > 1: the sample is cut into 2^20-parameter chunks that a pool of `threads` workers goes
    through (numpy releases the interpreter lock inside its loops): per chunk the mean gradient and its squared
    norm, then the clip coefficient from the sum, then per chunk AdamW; FedAvg per chunk likewise.  The sample's
    inputs come from the shared generator (filled on the GPU when there is one, since the fill is not what is
    being timed, then copied to the host).  Returns (params/s with FedAvg counted once per H steps, seconds of
    oracle work, threads)."""
    from oracle import fls_oracle as orc
    from concurrent.futures import ThreadPoolExecutor
    try:
        from threadpoolctl import threadpool_limits
    except Exception:                                   # pragma: no cover
        import contextlib
        threadpool_limits = lambda limits: contextlib.nullcontext()
    G, S, R = cfg["groups"], cfg["shard_dim"], cfg["replicate_dim"]
    K = S * R
    P = min(sample_params, cfg["n_params"])
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    f32 = cfg["grad_dtype"] == "f32"
    hp = orc.Hyper(cfg["lr"], cfg["beta1"], cfg["beta2"], cfg["eps"], cfg["weight_decay"], cfg["max_grad_norm"])
    th0 = sy.normal_fill_(torch.empty(P, device=dev), sy.stream_key(cfg["seed"], sy.KIND_MASTER), cfg["master_sigma"]).cpu().numpy()
    states = [orc.GroupState(th0.copy(), np.zeros(P, np.float32), np.zeros(P, np.float32), None) for _ in range(G)]
    raw = []
    for g in range(G):
        row = []
        for k in range(K):
            scale = sy.uniform_scale(cfg["seed"], g, k) if cfg["per_buffer_scale"] else 1.0
            t = sy.normal_fill_(torch.empty(P, dtype=torch.float32 if f32 else torch.bfloat16, device=dev),
                                sy.stream_key(cfg["seed"], sy.KIND_GRAD, 1, g, k), cfg["grad_sigma"], scale).cpu()
            row.append(t.numpy() if f32 else t.view(torch.int16).numpy().view(np.uint16))
        raw.append(row)
    counts = [sy.sample_count(cfg["seed"], g) for g in range(G)] if cfg["weights"] == "counts" else None
    as_f64 = (lambda x: x.astype(np.float64)) if f32 else orc.bf16_bits_to_f64
    with threadpool_limits(limits=1):
        if threads <= 1:
            t0 = time.perf_counter()
            for g in range(G):
                grads = [as_f64(x) for x in raw[g]]
                orc.sync_step_group(states[g], grads, S, R, 1, hp)
                del grads
            t_step = time.perf_counter() - t0
            t0 = time.perf_counter()
            orc.fedavg(states, counts)
            t_avg = time.perf_counter() - t0
        else:
            chunk = 1 << 20
            los = list(range(0, P, chunk))
            bits = [np.zeros(P, np.uint16) for _ in range(G)]
            with ThreadPoolExecutor(threads) as ex:
                t0 = time.perf_counter()
                for g in range(G):
                    st = states[g]
                    def reduce_chunk(lo, g=g):
                        gb = orc.reduce_mean([as_f64(x[lo:lo + chunk]) for x in raw[g]], S, R)
                        return gb, orc.grad_norm(gb) ** 2
                    parts = list(ex.map(reduce_chunk, los))
                    c = orc.clip_coef(float(np.sqrt(sum(sq for _, sq in parts))), hp.max_grad_norm)
                    def adamw_chunk(i, st=st, g=g):
                        lo = los[i]
                        sl = slice(lo, lo + chunk)
                        st.theta[sl], st.m[sl], st.v[sl], bits[g][sl] = orc.adamw(
                            st.theta[sl], st.m[sl], st.v[sl], parts[i][0], c, 1, hp.lr, hp.beta1, hp.beta2, hp.eps, hp.weight_decay)
                    list(ex.map(adamw_chunk, range(len(los))))
                    del parts
                t_step = time.perf_counter() - t0
                t0 = time.perf_counter()
                w = orc.fedavg_weights(counts, G)
                avg = np.empty(P, np.float32)
                def fedavg_chunk(lo):
                    sl = slice(lo, lo + chunk)
                    avg[sl] = orc.fedavg_array([st.theta[sl] for st in states], w)
                    bits[0][sl] = orc.f32_to_bf16_bits(avg[sl])
                list(ex.map(fedavg_chunk, los))
                for st in states:
                    st.theta[:] = avg
                t_avg = time.perf_counter() - t0
    sec = t_step + t_avg / cfg["sync_period"]
    return G * P / sec, t_step + t_avg, max(1, threads)


def sample_text(cfg: dict, n: int) -> str:
    return f"one oracle step of all {cfg['groups']} groups + FedAvg/H on the first {min(n, cfg['n_params'])} params of every buffer"


def cpu_baseline(cfg: dict) -> dict:
    """The oracle on this machine's host cores: all of them (the headline figure of this object), and one."""
    cores = host_cores()
    v1, s1, _ = oracle_sample(cfg, ORACLE_SAMPLE_ONE_CORE, 1)
    va, sa, used = oracle_sample(cfg, ORACLE_SAMPLE_ALL_CORES, cores)
    return {"value": va, "unit": UNIT, "cores": used, "kind": "oracle", "seconds": sa, "sample": sample_text(cfg, ORACLE_SAMPLE_ALL_CORES),
            "host_cores": cores,
            "one_core": {"value": v1, "unit": UNIT, "cores": 1, "seconds": s1, "sample": sample_text(cfg, ORACLE_SAMPLE_ONE_CORE)}}


def run_reference(args, cfg):
    """The reference arm of this build is the CPU oracle (the paper ships no code): every "step" is one
    oracle step + FedAvg/H on a bounded sample of the workload, on all host cores.  Rank 0 only."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = host_cores()
    vals, secs = [], []
    if args.warmup:
        oracle_sample(cfg, 1 << 18, cores)
    n = max(1, min(args.steps, 3))
    for _ in range(n):
        v, s, used = oracle_sample(cfg, ORACLE_SAMPLE_ALL_CORES, cores)
        vals.append(v); secs.append(s)
    value = float(np.mean(vals))
    v1, s1, _ = oracle_sample(cfg, ORACLE_SAMPLE_ONE_CORE, 1)
    what = sample_text(cfg, ORACLE_SAMPLE_ALL_CORES)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": n,
            "warmup": 1 if args.warmup else 0, "ms_per_step": 1e3 * float(np.mean(secs)), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": cfg["name"], "sample": what},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": used, "kind": "oracle", "sample": what, "host_cores": cores,
                             "one_core": {"value": v1, "unit": UNIT, "cores": 1, "seconds": s1,
                                          "sample": sample_text(cfg, ORACLE_SAMPLE_ONE_CORE)}},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------- GPU leg
def fill_session(sess, cfg):
    th_key = sy.stream_key(cfg["seed"], sy.KIND_MASTER)
    for g in range(cfg["groups"]):
        sy.normal_fill_(sess.master[g], th_key, cfg["master_sigma"])
        sess.param_bf16[g].copy_(sess.master[g])
        for k in range(sess.K):
            scale = sy.uniform_scale(cfg["seed"], g, k) if cfg["per_buffer_scale"] else 1.0
            sy.normal_fill_(sess.grads[g][k], sy.stream_key(cfg["seed"], sy.KIND_GRAD, 1, g, k), cfg["grad_sigma"], scale)
    torch.cuda.synchronize()


def measure_workload(args, cfg, fls, Session, rank, world, local, with_e2e, sampler):
    """Times one workload on this rank's GPU: K steps with events around the whole region, K more with events
    around every launch (per-kernel durations), optionally the end-to-end form with host gradients.  Returns the
    fields of the JSON line that describe this workload (rank 0) or None (other ranks)."""
    import torch.distributed as dist
    G, P = cfg["groups"], cfg["n_params"]
    counts = [sy.sample_count(cfg["seed"], g) for g in range(G)] if cfg["weights"] == "counts" else None
    fused = not args.unfused and G <= fls.FLS_MAX_FUSED_GROUPS
    sess = Session(P, cfg["unit_numel"], G, cfg["shard_dim"], cfg["replicate_dim"], cfg["sync_period"], cfg["grad_dtype"], 8,
                   args.opt_state, cfg["lr"], cfg["beta1"], cfg["beta2"], cfg["eps"], cfg["weight_decay"], cfg["max_grad_norm"],
                   device=f"cuda:{local}", fused=fused, speculative=args.speculative)
    H = cfg["sync_period"]
    for kern, val in (("reduce", args.ctas_reduce), ("adamw", args.ctas_adamw), ("fedavg", args.ctas_fedavg)):
        if val:
            fls.fls_plan_tune(sess.plan, {"reduce": 0, "adamw": 1, "fedavg": 2}[kern], val, -1)
    if args.descending_adamw:
        fls.fls_plan_tune(sess.plan, fls.FLS_KERNEL_ADAMW, 0, 1)
    if args.ascending_adamw:
        fls.fls_plan_tune(sess.plan, fls.FLS_KERNEL_ADAMW, 0, 0)
    if args.no_overlap:
        fls.fls_plan_set_overlap(sess.plan, False)
    if args.l2_keep_mb is not None:
        fls.fls_plan_set_l2_keep(sess.plan, int(args.l2_keep_mb * 2 ** 20))
    if args.batching is not None:
        fls.fls_plan_set_batching(sess.plan, args.batching)
    if args.resident is not None:
        fls.fls_plan_set_resident(sess.plan, args.resident)
    fill_session(sess, cfg)
    stream = torch.cuda.current_stream()

    n_fedavg = [0]

    def one_step():
        # on the steps where aggregation is due, the fused call does the step and FedAvg in one go
        if fused and (sess.t + 1) % H == 0:
            sess.step_fedavg(counts, stream=stream)
            n_fedavg[0] += 1
        elif sess.step(stream=stream):
            sess.fedavg(counts, stream=stream)
            n_fedavg[0] += 1

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    # Inputs larger than L2 need no flush.  A workload whose buffers fit in twice the L2 is timed step by step
    # with a write of a 512 MB buffer (untimed) before every step, so that no step starts with its inputs cached.
    eg = 4 if cfg["grad_dtype"] == "f32" else 2
    footprint = G * sess.n_padded * (sess.K * eg + 14) + 4 * sess.n_padded
    flush_buf = torch.empty(512 << 20, dtype=torch.uint8, device="cuda") if footprint < 2 * 126e6 else None

    def timed(n_steps, profiling, smp=None):
        fls.fls_set_profiling(sess.plan, profiling)
        barrier()
        l0 = fls.fls_get_launch_count(sess.plan)
        n_fedavg[0] = 0
        if flush_buf is None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(n_steps):
                one_step()
            e1.record(stream)
            if smp is not None:
                smp.wait_for(e1)
            barrier()
            ms = e0.elapsed_time(e1)
        else:
            ms = 0.0
            for i in range(n_steps):
                flush_buf.fill_(i & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream)
                one_step()
                e1.record(stream)
                if smp is not None:
                    smp.wait_for(e1)
                torch.cuda.synchronize()
                ms += e0.elapsed_time(e1)
            barrier()
        ms = max_over_ranks(ms, world, "cuda")
        return ms, fls.fls_get_launch_count(sess.plan) - l0

    for _ in range(args.warmup):
        one_step()
    ms_total, launches = timed(args.steps, False, sampler)
    fedavg_calls = n_fedavg[0]
    in_region = len(sampler.sm) if sampler is not None else 0
    # second pass over the same number of steps with events around every kernel: per-kernel durations
    # (the clocks keep being sampled: an NVML reading can take as long as a short timed region)
    ms_prof, _ = timed(args.steps, True, sampler)
    resident = fls.fls_plan_get_resident(sess.plan)
    batched = fls.fls_plan_get_batching(sess.plan) and not resident
    kms, kn = fls.fls_get_kernel_ms(sess.plan)
    fls.fls_set_profiling(sess.plan, False)
    spec = None
    if args.speculative:
        kept, redone = sess.spec_stats()          # all group-steps so far: warm-up, timed and profiled passes
        spec = {"group_steps_kept": kept, "group_steps_redone": redone, "hit_rate": kept / max(1, kept + redone)}

    # end to end: gradients start in pinned host memory, norms come back to the host, every step
    e2e = None
    h2d = G * sess.K * sess.n_padded * eg
    if with_e2e and h2d > args.e2e_max_gb * 2 ** 30:
        e2e = {"value": None, "unit": UNIT, "skipped": f"pinned host buffers above --e2e-max-gb {args.e2e_max_gb}"}
    elif with_e2e:
        try:
            host = [[torch.empty(sess.n_padded, dtype=sess.grad_torch_dtype, pin_memory=True) for _ in range(sess.K)] for _ in range(G)]
        except RuntimeError as err:                  # the host cannot pin that much memory: say so instead of failing the run
            host = None
            e2e = {"value": None, "unit": UNIT, "skipped": f"pinned host buffers of {h2d} bytes could not be allocated: {str(err)[:120]}"}
    if with_e2e and e2e is None:
        for g in range(G):
            for k in range(sess.K):
                host[g][k].copy_(sess.grads[g][k])
        norms = torch.zeros(G, dtype=torch.float32).pin_memory()
        def e2e_step():
            if sess.step_host(host, stream=stream, host_norms=norms):
                sess.fedavg(counts, stream=stream)
                torch.cuda.synchronize()
        e2e_step()
        barrier()
        t0 = time.perf_counter()
        n_e2e = max(2, min(args.steps, 4))
        for _ in range(n_e2e):
            e2e_step()
        torch.cuda.synchronize()
        dt = max_over_ranks(time.perf_counter() - t0, world, "cuda")
        e2e = {"value": world * G * P * n_e2e / dt, "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": 4 * G, "steps": n_e2e, "ms_per_step": 1e3 * dt / n_e2e}
        del host

    out = None
    if rank == 0:
        peak, peak_kind = measured_peak_gbs()
        N = sess.n_padded
        kbytes = sess.K * eg
        # FedAvg runs one launch per averaged array: parameters move 10 B per group-element (4 read, 4 + 2
        # written), m and v 8 B each; the figure is the mean over the launches of one call
        per_launch = {"reduce": N * (kbytes + 4), "adamw": N * 30, "fedavg": N * G * (26 / 3 if args.opt_state else 10),
                      "adamw_fedavg": N * G * 30}
        traffic_key = {"reduce": ("reduce", kbytes), "adamw": ("adamw", None), "fedavg": ("fedavg", None), "adamw_fedavg": ("adamw_fedavg", None)}
        units = {"reduce": N, "adamw": N, "fedavg": N * G, "adamw_fedavg": N * G}
        if not cfg["max_grad_norm"] > 0:
            # no clipping: one kernel per group does the whole step (timed under "adamw")
            per_launch.update(adamw=N * (kbytes + 26))
            traffic_key.update(adamw=("step_noclip", kbytes))
        elif kbytes < 8:
            # small K: nothing is stored by the norm pass and AdamW reads the gradients again
            per_launch.update(reduce=N * kbytes, adamw=N * (kbytes + 26))
            traffic_key.update(reduce=("norm_only", kbytes), adamw=("reduce_adamw", kbytes))
        if spec is not None:
            # two launches per group-step, both timed under "adamw": the guessing kernel always moves K*e_g + 26 B per
            # element, the follow-up kernel nothing when the guess held and the same again when it redoes the step
            per_launch.update(adamw=N * (kbytes + 26) * (1 + 1 - spec["hit_rate"]) / 2)
            traffic_key.update(adamw=("step_noclip", kbytes))
        if resident:
            # one cooperative kernel per step does everything for all groups (timed under "adamw")
            per_launch.update(adamw=G * N * (kbytes + 26))
            traffic_key.update(adamw=("step_resident", kbytes))
            units.update(adamw=N * G)
        if batched:
            # all groups in one grid: a reduce or AdamW launch covers G times the elements
            per_launch.update(reduce=G * per_launch["reduce"], adamw=G * per_launch["adamw"])
            units.update(reduce=N * G, adamw=N * G)
        kernels = {}
        for i, name in enumerate(("reduce", "adamw", "fedavg", "adamw_fedavg")):
            if kn[i]:
                avg_ms = kms[i] / kn[i]
                per_elem = NCU_TRAFFIC_BYTES_PER_ELEM.get(traffic_key[name])
                kernels[name] = {"launches": kn[i], "avg_ms": avg_ms, "bytes_per_launch": per_launch[name],
                                 "gbs": per_launch[name] / avg_ms / 1e6, "frac": per_launch[name] / avg_ms / 1e6 / peak,
                                 "frac_of_8tbs": per_launch[name] / avg_ms / 1e6 / 8000.0,
                                 "share": kms[i] / sum(kms), "traffic": per_elem * units[name] if per_elem else None}
        dom = max(kernels, key=lambda n: kernels[n]["share"])
        rep = fls.fls_comm_report(sess.plan)
        # bytes the timed steps had to move: every sync step, plus the FedAvg calls that fell inside the region
        # (the fused aggregation moves no bytes of its own: an aggregation step costs what a plain step costs)
        # (a resident plan's fused call is the resident step followed by a FedAvg kernel of its own)
        step_bytes = rep["hbm_bytes_sync_step"] + (0 if fused and not resident else rep["hbm_bytes_fedavg"] * fedavg_calls / args.steps)
        if spec is not None:
            step_bytes += rep["hbm_bytes_sync_step"] * (1 - spec["hit_rate"])       # a redone group-step moves its bytes twice
        ms_step = ms_total / args.steps
        out = {
            "value": world * G * P * args.steps / (ms_total / 1e3), "ms_per_step": ms_step,
            "config": {"workload": cfg["name"], "n_params": P, "groups": G, "shard_dim": cfg["shard_dim"],
                       "replicate_dim": cfg["replicate_dim"], "sync_period": cfg["sync_period"], "grad_dtype": cfg["grad_dtype"],
                       "fedavg_opt_state": bool(args.opt_state), "fused_aggregation": bool(fused), "groups_share_a_grid": bool(batched), "resident_step": bool(resident),
                       "fedavg_calls_in_timed_region": fedavg_calls,
                       "l2": "working set exceeds L2, no flush needed" if flush_buf is None else "L2 flushed (512 MB write, untimed) before every timed step",
                       "parallelism": "replicas only" if world > 1 else "1 gpu"},
            "hbm_gbs": step_bytes / ms_step / 1e6, "hbm_frac_of_measured_peak": step_bytes / ms_step / 1e6 / peak,
            "hbm_frac_of_8tbs": step_bytes / ms_step / 1e6 / 8000.0,
            "roofline": {"bound": "hbm", "kernel": dom, "achieved": kernels[dom]["gbs"], "peak": peak, "peak_kind": peak_kind,
                         "unit": "GB/s", "frac": kernels[dom]["frac"], "traffic": kernels[dom]["traffic"]},
            "kernels": kernels, "ms_per_step_profiled": ms_prof / args.steps,
            "gpu_launches": launches, "samples_in_timed_region": in_region, "e2e": e2e,
        }
        if spec is not None:
            out["config"]["speculative_single_pass"] = spec
    sess.close()
    del sess, flush_buf
    torch.cuda.empty_cache()
    return out


def run_ours(args, cfg):
    import torch.distributed as dist
    from paper_2609_20359_b200 import build

    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    # only now: importing the binding loads libfls.so, which rank 0 may just have built
    from paper_2609_20359_b200 import _binding as fls
    from paper_2609_20359_b200.session import Session

    sampler = ClockSampler(local) if rank == 0 else None
    if sampler is not None:
        sampler.start()
    main = measure_workload(args, cfg, fls, Session, rank, world, local, not args.no_e2e, sampler)
    others = {}
    if args.others:
        # the other two workloads of the target list, device-resident timing only; every rank runs them so that the
        # barriers match, rank 0 reports them
        for name in OTHER_WORKLOADS:
            if name == cfg["name"]:
                continue
            try:
                r = measure_workload(args, sy.config_by_name(name), fls, Session, rank, world, local, False, sampler)
            except (RuntimeError, MemoryError) as err:     # e.g. not enough free HBM: the main line must still be printed
                if world > 1:
                    raise                                   # the ranks' barriers would no longer match
                others[name] = {"error": str(err)[:200]}
                torch.cuda.empty_cache()
                continue
            if r is not None:
                others[name] = {k: r[k] for k in ("value", "ms_per_step", "hbm_gbs", "hbm_frac_of_measured_peak", "hbm_frac_of_8tbs",
                                                  "roofline", "kernels", "gpu_launches", "config")}
    if rank == 0:
        clocks = sampler.stop()
        clocks["samples_in_timed_region"] = main.pop("samples_in_timed_region")
        line = {"metric": METRIC, "value": main["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
                "ms_per_step": main["ms_per_step"], "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic"}
        line.update({k: v for k, v in main.items() if k not in ("value", "ms_per_step")})
        line["clocks"] = clocks
        if others:
            line["other_workloads"] = others
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(cfg)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------- launching N ranks
def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(n: int, argv) -> int:
    """`--gpus N` without a launcher: run this same command as N ranks, one process per GPU, under
    torch.distributed.run on this node.  Returns the launcher's exit code."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.run(cmd).returncode


def run_stub(args):
    """Launch plumbing without a GPU (used by the CPU tests): every rank "times" a step whose duration depends on
    its rank, the ranks agree on the slowest over gloo, rank 0 prints the line."""
    import torch.distributed as dist
    rank, world = int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks(10.0 * (rank + 1) * args.steps, world)
    units = 1000
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": world * units * args.steps / (ms / 1e3), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                          "config": {"workload": "stub", "parallelism": "replicas only" if world > 1 else "1 gpu"}}), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------- bandwidth sweep
SWEEP_SPLITS = [(2, 1), (2, 2), (2, 4), (4, 4), (4, 8), (8, 8)]       # (G, K): R*G = 2, 4, 8, 16, 32, 64


def sweep_points(p_exps=(20, 22, 24, 26, 28, 30)):
    for e in p_exps:
        for G, K in SWEEP_SPLITS:
            for order in ("fsdp", "hsdp"):
                if order == "hsdp" and K < 2:
                    continue
                for dt in ("bf16", "f32"):
                    S, R = (K, 1) if order == "fsdp" else (K // 2, 2)
                    yield dict(P=1 << e, G=G, K=K, S=S, R=R, order=order, dtype=dt)


def run_sweep(args):
    """HBM GB/s of the fused reduce+AdamW step and of FedAvg over flat P = 2^20 .. 2^30, R*G in 2..64,
    FL+FSDP vs FL+HSDP order, bf16 vs fp32 gradients.  One JSON line per point into --sweep-out.  Points whose
    buffers would not fit in 90 % of the free HBM are reported as skipped; points whose working set is below
    twice the L2 get an L2 flush (a 512 MB write) before every timed call."""
    from paper_2609_20359_b200 import build
    from paper_2609_20359_b200 import _binding as fls
    from paper_2609_20359_b200.session import Session
    build.build()
    torch.cuda.set_device(0)
    peak, peak_kind = measured_peak_gbs()
    flush = torch.empty(512 << 20, dtype=torch.uint8, device="cuda")
    block = 1 << 22
    seedbuf = {dt: sy.normal_fill_(torch.empty(block, dtype=torch.float32 if dt == "f32" else torch.bfloat16, device="cuda"),
                                   sy.stream_key(5, sy.KIND_GRAD, 1, 0, 0), 1e-3) for dt in ("bf16", "f32")}
    seedth = sy.normal_fill_(torch.empty(block, device="cuda"), sy.stream_key(5, sy.KIND_MASTER), 0.02)
    out = open(args.sweep_out, "w")
    exps = [int(x) for x in args.sweep_exps.split(",")]
    for pt in sweep_points(exps):
        P, G, K = pt["P"], pt["G"], pt["K"]
        eg = 4 if pt["dtype"] == "f32" else 2
        need = G * K * P * eg + G * 14 * P + 4 * P + (64 << 20)
        free, _ = torch.cuda.mem_get_info()
        rec = dict(pt, bytes_needed=need)
        if need > 0.9 * free:
            rec["skipped"] = "exceeds HBM"
            out.write(json.dumps(rec) + "\n"); out.flush()
            continue
        sess = Session(P, None, G, pt["S"], pt["R"], 1, pt["dtype"], 8, False)
        if args.batching is not None and (args.batching <= 0 or G > 1):
            try:
                fls.fls_plan_set_batching(sess.plan, args.batching)
            except fls.FlsError:
                pass                                   # forcing it on a shape that has no shared-grid form
        if args.resident is not None and args.resident <= 0:
            fls.fls_plan_set_resident(sess.plan, args.resident)
        for g in range(G):
            # the fill repeats a 4 Mi-element generator block (bandwidth does not depend on the values)
            for buf, src in [(sess.master[g], seedth)] + [(b, seedbuf[pt["dtype"]]) for b in sess.grads[g]]:
                n = buf.numel()
                if n >= block:
                    buf[: n // block * block].view(-1, block).copy_(src.expand(n // block, block))
                buf[n // block * block:].copy_(src[: n % block])
        torch.cuda.synchronize()
        resident = need < 2 * 126e6
        stream = torch.cuda.current_stream()
        def timed(call, reps):
            ts = []
            for i in range(reps + 3):
                if resident:
                    flush.fill_(i & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record(stream); call(); e1.record(stream)
                torch.cuda.synchronize()
                if i >= 3:
                    ts.append(e0.elapsed_time(e1))
            return float(np.median(ts))
        ms_step = timed(lambda: sess.step(stream=stream), 5)
        ms_avg = timed(lambda: sess.fedavg(None, stream=stream), 3)
        rep = fls.fls_comm_report(sess.plan)
        rec.update(ms_sync_step=ms_step, ms_fedavg=ms_avg, l2_flush=resident,
                   sync_step_gbs=rep["hbm_bytes_sync_step"] / ms_step / 1e6, fedavg_gbs=rep["hbm_bytes_fedavg"] / ms_avg / 1e6,
                   synced_params_per_s=G * P / (ms_step / 1e3))
        rec["sync_step_frac_of_8tbs"] = rec["sync_step_gbs"] / 8000.0
        rec["fedavg_frac_of_8tbs"] = rec["fedavg_gbs"] / 8000.0
        rec["peak_gbs"], rec["peak_kind"] = peak, peak_kind
        out.write(json.dumps(rec) + "\n"); out.flush()
        sess.close()
        del sess
        torch.cuda.empty_cache()
    out.close()
    print(json.dumps({"sweep": args.sweep_out}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=16)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default=DEFAULT_CONFIG, choices=[c["name"] for c in sy.CONFIGS])
    ap.add_argument("--opt-state", action="store_true", help="FedAvg also averages m and v")
    ap.add_argument("--unfused", action="store_true", help="aggregation steps call fls_sync_step + fls_fedavg instead of fls_sync_step_fedavg")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--e2e-max-gb", type=float, default=48.0, help="skip the end-to-end pass if its pinned host staging would exceed this")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-others", dest="others", action="store_false", help="time only the chosen workload (default: the default workload is followed by the other two target workloads)")
    ap.add_argument("--stub-workload", action="store_true", help=argparse.SUPPRESS)   # launch plumbing on CPU, for the tests
    ap.add_argument("--ctas-reduce", type=int, default=0)
    ap.add_argument("--ctas-adamw", type=int, default=0)
    ap.add_argument("--ctas-fedavg", type=int, default=0)
    ap.add_argument("--descending-adamw", action="store_true")
    ap.add_argument("--ascending-adamw", action="store_true")
    ap.add_argument("--no-overlap", action="store_true", help="plain launches instead of programmatic dependent launch")
    ap.add_argument("--speculative", action="store_true", help="speculative single pass (guess: clip coefficient 1) with a second set of state buffers")
    ap.add_argument("--batching", type=int, default=None, choices=[-1, 0, 1], help="all groups in one grid per kernel: -1 automatic (small plans), 0 never, 1 whenever possible")
    ap.add_argument("--resident", type=int, default=None, choices=[-1, 0, 1], help="whole step of all groups as one cooperative kernel: -1 automatic (small plans), 0 never, 1 whenever the plan fits the device")
    ap.add_argument("--l2-keep-mb", type=float, default=None, help="MiB at the end of the reduced gradient stored with L2 evict-last (library default: 64)")
    # slices of a workload, for profiler captures that must stay small (same kernels, fewer bytes)
    ap.add_argument("--n-params", type=int, default=0, help="override P (single flat unit)")
    ap.add_argument("--groups", type=int, default=0, help="override G")
    ap.add_argument("--sync-period", type=int, default=0, help="override H")
    ap.add_argument("--shard-dim", type=int, default=0, help="override S")
    ap.add_argument("--replicate-dim", type=int, default=0, help="override R_rep")
    ap.add_argument("--grad-dtype", default="", choices=["", "bf16", "f32"], help="override the gradient dtype")
    ap.add_argument("--keep-units", action="store_true", help="with --n-params: keep the unit table's proportions")
    ap.add_argument("--clip", type=float, default=None, help="override max_grad_norm (0 disables clipping: single-pass step)")
    ap.add_argument("--sweep", action="store_true", help="run the bandwidth sweep instead of the benchmark")
    ap.add_argument("--sweep-out", default="sweep_results.jsonl")
    ap.add_argument("--sweep-exps", default="20,22,24,26,28,30", help="log2 of the parameter counts to sweep")
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started without a launcher: become N ranks
        raise SystemExit(spawn_ranks(args.gpus, sys.argv[1:]))
    if args.stub_workload:
        run_stub(args)
        return
    if args.sweep:
        os.makedirs(os.path.dirname(args.sweep_out) or ".", exist_ok=True)
        run_sweep(args)
        return
    cfg = sy.config_by_name(args.config)
    sliced = any([args.n_params, args.groups, args.sync_period, args.shard_dim, args.replicate_dim, args.clip is not None, args.grad_dtype])
    if sliced or args.config != DEFAULT_CONFIG or args.speculative:
        args.others = False
    if args.n_params and args.keep_units:
        # same unit table, every unit scaled by n_params / P and rounded to a multiple of 64 elements
        units = [max(64, int(round(u * args.n_params / cfg["n_params"] / 64)) * 64) for u in cfg["unit_numel"]]
        cfg.update(n_params=sum(units), unit_numel=units, name=cfg["name"] + f"[P={sum(units)}, {len(units)} units]")
    elif args.n_params:
        cfg.update(n_params=args.n_params, unit_numel=[args.n_params], name=cfg["name"] + f"[P={args.n_params}]")
    if args.groups:
        cfg.update(groups=args.groups, name=cfg["name"] + f"[G={args.groups}]")
    if args.sync_period:
        cfg.update(sync_period=args.sync_period, name=cfg["name"] + f"[H={args.sync_period}]")
    if args.shard_dim:
        cfg.update(shard_dim=args.shard_dim, name=cfg["name"] + f"[S={args.shard_dim}]")
    if args.replicate_dim:
        cfg.update(replicate_dim=args.replicate_dim, name=cfg["name"] + f"[R={args.replicate_dim}]")
    if args.clip is not None:
        cfg.update(max_grad_norm=args.clip, name=cfg["name"] + f"[clip={args.clip}]")
    if args.grad_dtype:
        cfg.update(grad_dtype=args.grad_dtype, name=cfg["name"] + f"[{args.grad_dtype}]")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Throughput of the batched verify-and-resample round of Cool-SD on B200.

A "step" is one call of the whole path (row statistics, relaxed acceptance test, first
rejection, optimal resampling distribution, inverse-CDF draw, emit) over one batch of
synthetic logits.  Default workload: B=64 sequences x gamma=8 drafted positions x V=16384
image tokens, bf16 logits, conditional/unconditional rows mixed on load (scale 4) and top-k
1000 before the softmax, annealed schedule delta=1.1, nu=0.7.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference] [--workload C3]

One JSON line on stdout (rank 0).  `value` is verified draft tokens per second with the inputs
resident in HBM (a ring of distinct step inputs larger than L2, replayed as a CUDA graph; the timed
region is always whole replays -- at least max(K, 2048) calls per repetition, 7 repetitions, the
median reported -- so the figure does not depend on K); `stream_order` is the same call in
ordinary stream order, one call at a time, as a decoding loop issues it;
`e2e` is the same metric through the host-buffer entry point, host->device and device->host
copies inside the timed region; `roofline` compares the step's algorithmic bytes with the
measured HBM copy bandwidth; `cpu_baseline` is the fp64 CPU oracle timed on a bounded sample.
With N > 1 every rank runs the same batch shape on its own GPU (sequences are independent: no
exchange step, weak scaling).  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

MIN_TIMED_CALLS = 2048   # calls per timed repetition, at least (whole graph replays)
REPS = 7                 # timed repetitions; the median is reported
METRIC = "verified_draft_tokens_per_sec"
UNIT = "tokens/s"
L2_BYTES = 126 * 1024 * 1024
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# DRAM traffic of one launch of the dominant kernel (dram__bytes_read.sum + dram__bytes_write.sum,
# one ncu capture of this workload).  Reported only while the kernel sources still have the digest
# the capture was taken with; null otherwise.
NCU_TRAFFIC = {"sources_sha256": "3ee3f9f359ad5dd8", "workload": "C3", "bytes_per_launch": 68073984}


def sources_digest() -> str:
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2601_09212_b200", "csrc")
    for name in sorted(os.listdir(d)):
        with open(os.path.join(d, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks: NVML polled from a thread while the timed region runs (reading only)
class ClockSampler:
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown"}

    def __init__(self, pci_bus_id: str, period_s: float = 0.002):
        self.index, self.period = pci_bus_id, period_s
        self.samples, self.reasons, self.power = [], set(), []
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByPciBusId(pci_bus_id.encode())
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None

    def sample_once(self):
        if self._nvml is None:
            return
        n = self._nvml
        try:
            self.samples.append(int(n.nvmlDeviceGetClockInfo(self._h, n.NVML_CLOCK_SM)))
            r = int(n.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            for bit, name in self.REASONS.items():
                if r & bit:
                    self.reasons.add(name)
            self.power.append(n.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_once()
            self._stop.wait(self.period)

    def start(self):
        if self._nvml is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self) -> dict:
        if self._nvml is None or not self.samples:
            return self._smi_fallback()
        return {"sm_mhz": int(np.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None, "source": "nvml"}

    def _smi_fallback(self) -> dict:
        try:
            out = subprocess.run(
                ["nvidia-smi", f"--id={self.index}", "--query-gpu=clocks.sm,clocks.max.sm,"
                 "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
                 "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap",
                 "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=20).stdout
            f = [x.strip() for x in out.strip().split(",")]
            names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
            return {"sm_mhz": int(f[0]), "sm_max_mhz": int(f[1]),
                    "reasons": [n for n, v in zip(names, f[2:6]) if v.lower().startswith("active")],
                    "samples": 1, "source": "nvidia-smi after the timed region"}
        except Exception as e:  # noqa: BLE001
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "source": f"unavailable: {e}"}


# ---------------------------------------------------------------------------------------------
def workload_kwargs(name: str) -> dict:
    """A named configuration (C1..C4) or a sweep point such as "B=64,gamma=8,V=16384,dtype=bf16"
    (optional keys: rho, law, cfg, cfg_scale, top_k)."""
    from paper_2601_09212_b200 import workloads as W
    if name in W.CONFIGS:
        kw = dict(W.CONFIGS[name])
        kw.pop("steps", None)
        return kw
    kw = dict(rho=0.9)
    for item in name.split(","):
        k, v = item.split("=")
        k = k.strip()
        if k == "dtype":
            kw[k] = {"bf16": W.BF16, "fp32": W.F32, "f32": W.F32}[v.strip()]
        elif k in ("B", "gamma", "V", "top_k"):
            kw[k] = int(v)
        elif k in ("rho", "cfg_scale", "scale"):
            kw[k] = float(v)
        elif k == "cfg":
            kw[k] = v.strip() in ("1", "true", "True")
        elif k == "law":
            kw[k] = v.strip()
        else:
            raise SystemExit(f"unknown workload key {k}")
    for need in ("B", "gamma", "V"):
        if need not in kw:
            raise SystemExit(f"workload needs {need}")
    return kw


def describe(name: str, kw: dict, sched_desc: str) -> dict:
    from paper_2601_09212_b200 import workloads as W
    d = {"workload": name, "B": kw["B"], "gamma": kw["gamma"], "V": kw["V"],
         "logits": "bf16" if kw.get("dtype", W.F32) == W.BF16 else "fp32",
         "guidance_mix": bool(kw.get("cfg", False)), "cfg_scale": kw.get("cfg_scale", 1.0) if kw.get("cfg") else None,
         "top_k": kw.get("top_k", 0), "rho": kw.get("rho"), "law": kw.get("law", "gauss"),
         "schedule": sched_desc, "target_rows": kw["gamma"]}
    return d


def algorithmic_bytes(kw: dict) -> int:
    """Bytes one step must move: every stored logit once, plus tokens, uniforms, schedule, outputs."""
    from paper_2601_09212_b200 import workloads as W
    e = 2 if kw.get("dtype", W.F32) == W.BF16 else 4
    A = 2 if kw.get("cfg") else 1
    B, L, V = kw["B"], kw["gamma"], kw["V"]
    return e * V * B * A * (L + L) + 4 * B * L + 4 * B * (L + 1) + 4 * L + 4 * B * (L + 2)


def oracle_schedule(L: int):
    import oracle
    return oracle.make_schedule(1, 1.1, 0.7, L).astype(np.float32)


def time_oracle(name: str, kw: dict, n_steps: int, seqs_per_step: int, warm: int = 0, seed: int = 0,
                device="cpu", ring: int = 4):
    """Times the CPU oracle as it stands on `n_steps` steps of `seqs_per_step` sequences each, drawn
    from a small ring of seeded batches with the workload's recipe (generated outside the timed
    region).  Returns (seconds, sequences processed, threads)."""
    import oracle
    from paper_2601_09212_b200 import workloads as W
    oracle.build()
    L = kw["gamma"]
    sched = oracle_schedule(L)
    kw = dict(kw, B=int(seqs_per_step))
    batches = []
    for s in range(min(ring, warm + n_steps)):
        w = W.make(name, seed=1000 + seed, step=s, schedule=sched, device=device, **kw)
        batches.append((w, w.host_arrays()))
    total_t, total_seq = 0.0, 0
    for s in range(warm + n_steps):
        w, h = batches[s % len(batches)]
        t0 = time.perf_counter()
        oracle.verify(h["target_logits"], h["draft_logits"], h["draft_tokens"], h["uniforms"],
                      h["relax_schedule"], dtype=w.dtype, target_uncond=h["target_uncond"],
                      draft_uncond=h["draft_uncond"], cfg_scale=w.cfg_scale, top_k=w.top_k,
                      want_G=False, want_pqf=False)
        dt = time.perf_counter() - t0
        if s >= warm:
            total_t += dt
            total_seq += int(seqs_per_step)
    return total_t, total_seq, oracle.num_threads()


def run_reference(args) -> None:
    """The CPU oracle as the reference arm: K timed steps, each a bounded sample of the workload
    (a batch of fewer sequences, same recipe), sized so that the run takes about two minutes."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    name = args.workload
    kw = workload_kwargs(name)
    oracle.build()
    threads = oracle.num_threads()
    L, B = kw["gamma"], kw["B"]
    side = min(B, threads)                     # sequences that run side by side, one per thread
    t_round, _, _ = time_oracle(name, kw, 1, side, warm=1)
    budget = 120.0
    rounds = max(1, int(budget / (args.steps + args.warmup) / max(t_round, 1e-6)))
    seqs = int(min(B, rounds * side))
    t, nseq, _ = time_oracle(name, kw, args.steps, seqs, warm=args.warmup)
    value = nseq * L / t
    sample = (f"{seqs} of {B} sequences per step, {args.steps} steps over a ring of 4 seeded batches "
              f"of the workload's recipe")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": describe(name, kw, "exp delta=1.1 nu=0.7"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
def run_native(args) -> None:
    import torch
    import paper_2601_09212_b200 as csd
    from paper_2601_09212_b200 import _build, sharding, workloads as W

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    _build.build_library()
    csd.library()

    name = args.workload
    kw = workload_kwargs(name)
    B, L, V, dtype = kw["B"], kw["gamma"], kw["V"], kw.get("dtype", W.F32)
    sched = csd.csd_make_schedule(1, 1.1, 0.7, L)
    step_bytes = algorithmic_bytes(kw)
    ring_n = max(4, -(-4 * L2_BYTES // step_bytes))          # ring of distinct inputs >= 4 x L2
    ring_n = min(ring_n, 64)
    ring = [W.make(name, seed=1 + rank, step=s, schedule=sched, device=dev, **kw) for s in range(ring_n)]
    outs = [dict(tok=torch.empty(B, L + 1, dtype=torch.int32, device=dev),
                 tau=torch.empty(B, dtype=torch.int32, device=dev),
                 st=torch.empty(B, dtype=torch.int32, device=dev),
                 am=torch.empty(B, L, device=dev) if args.monitors else None,
                 bt=torch.empty(B, L, device=dev) if args.monitors else None,
                 ws=csd.new_workspace(B, L, V, dtype, dev)) for _ in range(ring_n)]
    stream = torch.cuda.Stream(device=dev)
    prms = [csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                            o["tok"], o["tau"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                            cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=o["st"], workspace=o["ws"],
                            stream=stream, back_to_back=not args.single_call_latency,
                            diag_accept_mass=o["am"], diag_bound_term=o["bt"])
            for w, o in zip(ring, outs)]
    kernels_per_step = csd.csd_launch_count(prms[0])

    # The same calls in ordinary stream order (back_to_back = 0): what a decoding loop sees, whose logits
    # come from the forward pass just before the call.  Timed beside the headline, reported beside it.
    prms_so = [csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule,
                               o["tok"], o["tau"], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                               cfg_scale=w.cfg_scale, top_k=w.top_k, out_status=o["st"], workspace=o["ws"],
                               stream=stream, back_to_back=False,
                               diag_accept_mass=o["am"], diag_bound_term=o["bt"])
               for w, o in zip(ring, outs)]

    # A few laps of the ring as one CUDA graph: the launches inside are the library's own.  Inside a
    # graph consecutive calls keep their programmatic-launch edges and overlap as they do when enqueued
    # directly; two replays do not overlap, so the graph is made long enough (>= 64 calls) for that
    # boundary not to matter.  Whatever --steps is, the timed region is whole replays of that graph:
    # REPS repetitions of at least max(steps, MIN_TIMED_CALLS) calls each, each repetition between its
    # own pair of events; the reported time per step is the median repetition.
    graph_steps = ring_n * max(1, -(-64 // ring_n))

    def capture(params):
        with torch.cuda.stream(stream):
            for i in range(ring_n):
                csd.csd_verify_ex(params[i])
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for i in range(graph_steps):
                csd.csd_verify_ex(params[i % ring_n])
        return g

    graph = capture(prms)
    graph_so = capture(prms_so)
    replays = max(1, -(-max(args.steps, MIN_TIMED_CALLS) // graph_steps))
    replays_so = max(1, replays // 4)
    timed_calls = replays * graph_steps

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed_reps(g, n_replays, reps):
        """ms of each of `reps` repetitions of n_replays replays (max over ranks each)."""
        out = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            barrier()
            with torch.cuda.stream(stream):
                a.record(stream)
                for _ in range(n_replays):
                    g.replay()
                b.record(stream)
            barrier()
            out.append(sharding.max_over_ranks(a.elapsed_time(b), device=dev))
        return out

    warm_replays = max(1, -(-max(args.warmup, 3) // graph_steps))
    with torch.cuda.stream(stream):
        for _ in range(warm_replays):
            graph.replay()
            graph_so.replay()
    barrier()
    props = torch.cuda.get_device_properties(dev)
    sampler = ClockSampler(f"{props.pci_domain_id:08x}:{props.pci_bus_id:02x}:{props.pci_device_id:02x}.0")
    sampler.start()
    rep_ms = timed_reps(graph, replays, REPS)
    sampler.sample_once()
    sampler.stop()
    so_ms = timed_reps(graph_so, replays_so, 3)
    step_ms_reps = sorted(m / timed_calls for m in rep_ms)
    step_ms = float(np.median(step_ms_reps))
    so_step_ms = float(np.median(so_ms)) / (replays_so * graph_steps)
    with torch.cuda.stream(stream):   # leave the outputs of the headline mode in place for the checks below
        graph.replay()
    barrier()

    # accepted lengths of the last lap (a property of the synthetic drafter, reported for context)
    mean_emit = float(np.mean([o["tau"].float().mean().item() + 1.0 for o in outs]))

    # ---- end to end: host buffers in, host results out, copies inside the timed region ----------
    e2e_steps = max(1, min(args.steps, 48))
    host_n = 2
    pin = lambda t: None if t is None else t.cpu().pin_memory()
    hprm, hkeep = [], []
    for w in ring[:host_n]:
        hb = dict(t=pin(w.target_logits), d=pin(w.draft_logits), tu=pin(w.target_uncond), du=pin(w.draft_uncond),
                  tok=pin(w.draft_tokens), u=pin(w.uniforms), s=pin(w.relax_schedule),
                  ot=torch.empty(B, L + 1, dtype=torch.int32).pin_memory(),
                  ol=torch.empty(B, dtype=torch.int32).pin_memory(),
                  os=torch.empty(B, dtype=torch.int32).pin_memory())
        p = csd.make_params(hb["t"], hb["d"], hb["tok"], hb["u"], hb["s"], hb["ot"], hb["ol"],
                            target_uncond=hb["tu"], draft_uncond=hb["du"], cfg_scale=w.cfg_scale, top_k=w.top_k,
                            out_status=hb["os"], stream=stream, host=True)
        hprm.append(p)
        hkeep.append(hb)
    staging = [torch.empty(csd.csd_host_staging_size(p), dtype=torch.uint8, device=dev) for p in hprm]
    h2d = sum(t.numel() * t.element_size() for k, t in hkeep[0].items()
              if t is not None and k in ("t", "d", "tu", "du", "tok", "u", "s"))
    d2h = sum(hkeep[0][k].numel() * 4 for k in ("ot", "ol", "os"))
    for i in range(3):
        csd.csd_verify_host(hprm[i % host_n], staging[i % host_n])
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(e2e_steps):
        csd.csd_verify_host(hprm[i % host_n], staging[i % host_n])
    f1.record(stream)
    barrier()
    e2e_ms = sharding.max_over_ranks(f0.elapsed_time(f1), device=dev)
    # the host arrays now hold the last step's results; they must equal the device-resident run's
    last = (e2e_steps - 1) % host_n
    same = bool(np.array_equal(hkeep[last]["ot"].numpy(), outs[last]["tok"].cpu().numpy()))

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    value = sharding.job_throughput(B * L, world, step_ms * 1e-3)
    peak, peak_kind = measured_peak()
    step_s = step_ms * 1e-3
    achieved = step_bytes / step_s / 1e9
    so_achieved = step_bytes / (so_step_ms * 1e-3) / 1e9
    digest = sources_digest()
    traffic = None
    if (NCU_TRAFFIC["sources_sha256"] == digest and NCU_TRAFFIC["workload"] == name
            and not args.single_call_latency and not args.monitors):
        traffic = NCU_TRAFFIC["bytes_per_launch"]
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": step_ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": describe(name, kw, "exp delta=1.1 nu=0.7"),
        "timed_calls": timed_calls, "reps": REPS,
        "ms_per_step_reps": {"min": step_ms_reps[0], "median": step_ms, "max": step_ms_reps[-1]},
        "run": {"parallelism": f"dp{world} (independent sequences, no exchange)",
                "l2": f"ring of {ring_n} distinct step inputs, {ring_n * step_bytes / 1e6:.0f} MB > {L2_BYTES / 1e6:.0f} MB L2",
                "launch": f"CUDA graph of {graph_steps} calls, {replays} replays per repetition, {REPS} repetitions "
                          f"(median reported); warm-up {warm_replays} replays",
                "monitors": bool(args.monitors),
                "partition": ("one call at a time: ordinary stream order, sequences split over clusters" if args.single_call_latency
                              else "back_to_back: consecutive calls overlap (programmatic dependent launch)"),
                "arithmetic": "fp32 exponentials and sums, fp64 running sums in the draw; logits stored as "
                              + ("bf16" if dtype == W.BF16 else "fp32")},
        "clocks": sampler.summary(),
        "e2e": {"value": B * L * e2e_steps * world / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "entry": "csd_verify_host (pinned host buffers)",
                "matches_device_run": same},
        "gpu_launches": kernels_per_step * timed_calls * REPS,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": traffic, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS,
                     "bytes_per_launch": step_bytes,
                     "duration_us": step_s * 1e6,
                     "kernel": "the single fused launch of a step" if kernels_per_step == 1 else "all launches of a step",
                     "note": "duration = median repetition / its launches, CUDA events on the launching stream; calls "
                             "overlap, so this is the sustained time per launch"},
        "stream_order": {"us_per_call": so_step_ms * 1e3, "achieved": so_achieved, "unit": "GB/s", "frac": so_achieved / peak,
                         "calls": replays_so * graph_steps, "reps": 3,
                         "note": "back_to_back = 0: each call starts when the one before it has completed, as in a "
                                 "decoding loop whose logits come from the forward pass just before the call"},
        "emitted_tokens_per_step_mean": B * mean_emit,
    }
    if world == 1 and not args.no_cpu_baseline:
        t1, n1, threads = time_oracle(name, kw, 1, B, device=dev)
        n = int(min(64, max(1, round(12.0 / max(t1, 1e-3)))))
        t, nseq, threads = time_oracle(name, kw, n, B, seed=7, device=dev)
        import oracle
        oracle.set_num_threads(1)
        n_one = int(min(B, 8))   # one thread: a few sequences are a few seconds
        ts, ns, _ = time_oracle(name, kw, 1, n_one, seed=11, device=dev)
        oracle.set_num_threads(threads)
        line["cpu_baseline"] = {"value": nseq * L / t, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{n} full steps ({nseq} sequences, ring of 4 seeded batches) of the "
                                          f"same workload, {t:.1f} s wall",
                                "single_thread": {"value": ns * L / ts, "unit": UNIT, "cores": 1,
                                                  "sample": f"{ns} sequences of one step, {ts:.1f} s wall"}}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


def run_drafting_stage(args) -> None:
    """Side measurement (not the headline): csd_sample_rows on the drafter rows of the workload --
    R = B * gamma rows, one token each -- timed like the round: resident inputs larger than L2, a CUDA
    graph of 64 calls replayed, CUDA events on the launching stream.  One GPU."""
    import torch
    from paper_2601_09212_b200 import _build, workloads as W
    import paper_2601_09212_b200 as csd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    _build.build_library()
    name = args.workload
    kw = workload_kwargs(name)
    B, L, V, dtype = kw["B"], kw["gamma"], kw["V"], kw.get("dtype", W.F32)
    R = B * L
    arrays = 2 if kw.get("cfg") else 1
    step_bytes = R * V * (2 if dtype == W.BF16 else 4) * arrays + 8 * R
    ring_n = min(64, max(4, -(-4 * L2_BYTES // step_bytes)))
    sched = csd.csd_make_schedule(1, 1.1, 0.7, L)
    ring = [W.make(name, seed=1, step=s, schedule=sched, device=dev, **kw) for s in range(ring_n)]
    stream = torch.cuda.Stream(device=dev)
    calls = []
    for w in ring:
        calls.append(dict(
            logits=w.draft_logits.reshape(R, V), unc=None if w.draft_uncond is None else w.draft_uncond.reshape(R, V),
            uni=torch.rand(R, device=dev) * 0.999 + 0.0005, tok=torch.empty(R, dtype=torch.int32, device=dev),
            ws=torch.zeros(csd.csd_sample_workspace_size(R, V, dtype), dtype=torch.uint8, device=dev),
            scale=w.cfg_scale, k=w.top_k))

    def enqueue(i):
        c = calls[i % ring_n]
        csd.csd_sample_rows(c["logits"], c["uni"], c["tok"], uncond=c["unc"], cfg_scale=c["scale"], top_k=c["k"],
                            workspace=c["ws"], back_to_back=not args.single_call_latency, stream=stream)

    graph_steps = ring_n * max(1, -(-64 // ring_n))
    with torch.cuda.stream(stream):
        for i in range(ring_n):
            enqueue(i)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for i in range(graph_steps):
            enqueue(i)
    replays = max(1, args.steps // graph_steps)
    with torch.cuda.stream(stream):
        for _ in range(max(1, args.warmup // graph_steps)):
            graph.replay()
    stream.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        e0.record(stream)
        for _ in range(replays):
            graph.replay()
        e1.record(stream)
    stream.synchronize()
    steps = replays * graph_steps
    ms = e0.elapsed_time(e1)
    peak, peak_kind = measured_peak()
    achieved = step_bytes / (ms * 1e-3 / steps) / 1e9
    print(json.dumps({
        "metric": "sampled_draft_tokens_per_sec", "value": R * steps / (ms * 1e-3), "unit": "tokens/s", "n_gpus": 1,
        "steps": steps, "ms_per_step": ms / steps, "higher_is_better": True, "data": "synthetic",
        "config": dict(describe(name, kw, "-"), rows=R, op="csd_sample_rows (Algorithm 1, drafting stage)",
                       launch=f"CUDA graph of {graph_steps} calls, replayed"),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "bytes_per_launch": step_bytes, "traffic": None},
    }))


def run_widened(args) -> None:
    """Side measurements (not the headline) of the widened entry points on the workload's shapes: tree
    verification (csd_verify_tree, a static 4-3-2-2 tree), similarity-relaxed acceptance
    (csd_verify_similar, k = 10 neighbours, lambda = 2) and one rank's four calls of the
    vocabulary-sharded round (csd_shard_*, with the whole vocabulary or a quarter of it as the slice;
    the all-gathers are replaced by views of the rank's own buffers, so this is kernel time only).
    Timed like the round: resident inputs larger than L2, a CUDA graph of calls replayed, CUDA events on
    the launching stream, calls in stream order.  One GPU."""
    import numpy as np
    import torch
    from paper_2601_09212_b200 import _build, workloads as W
    import paper_2601_09212_b200 as csd
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    _build.build_library()
    kind, name = args.widened, args.workload
    kw = workload_kwargs(name)
    B, L, V, dtype = kw["B"], kw["gamma"], kw["V"], kw.get("dtype", W.F32)
    es = 2 if dtype == W.BF16 else 4
    arrays = 2 if kw.get("cfg") else 1
    stream = torch.cuda.Stream(device=dev)
    keep = []
    if kind == "tree":
        parent = W.static_tree([4, 3, 2, 2])
        N, D = len(parent), csd.csd_tree_depth(parent)
        sched = csd.csd_make_schedule(1, 1.1, 0.7, D)
        step_bytes = 2 * arrays * (N + 1) * V * es * B
        units, unit_name, op = B * N, "verified_tree_nodes_per_sec", f"csd_verify_tree, static tree 4-3-2-2 ({N} nodes, depth {D})"
        ring_n = max(2, -(-2 * L2_BYTES // step_bytes))
        tkw = {k: v for k, v in kw.items() if k not in ("B", "gamma", "V", "bonus_row")}
        for s_ in range(ring_n):
            w = W.make_tree(parent, B=B, V=V, schedule=sched, seed=1, step=s_, device=dev, **tkw)
            out = (torch.empty(B, D + 1, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev))
            ws = torch.zeros(csd.csd_tree_workspace_size(B, N, V, dtype), dtype=torch.uint8, device=dev)
            keep.append((w, out, ws))

        def enqueue(i):
            w, out, ws = keep[i % ring_n]
            csd.csd_verify_tree(w.target_logits, w.draft_logits, w.parent, w.draft_tokens, w.uniforms, w.relax_schedule,
                                out[0], out[1], target_uncond=w.target_uncond, draft_uncond=w.draft_uncond,
                                cfg_scale=w.cfg_scale, top_k=w.top_k, workspace=ws, stream=stream)

    elif kind == "similar":
        sched = csd.csd_make_schedule(1, 1.1, 0.7, L)
        step_bytes = algorithmic_bytes(kw)
        units, unit_name, op = B * L, "verified_draft_tokens_per_sec", "csd_verify_similar, k = 10 neighbours, lambda = 2"
        ring_n = max(2, -(-2 * L2_BYTES // step_bytes))
        r = np.random.default_rng(5)
        nb = ((np.arange(V)[:, None] + 1 + r.integers(0, V - 1, size=(V, 10))) % V).astype(np.int32)   # never the token itself
        table = torch.from_numpy(nb).to(dev)
        for s_ in range(ring_n):
            w = W.make(name, seed=1, step=s_, schedule=sched, device=dev, **kw)
            out = (torch.empty(B, L + 1, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev))
            ws = csd.new_workspace(B, L, V, dtype, dev)
            prm = csd.make_params(w.target_logits, w.draft_logits, w.draft_tokens, w.uniforms, w.relax_schedule, out[0], out[1],
                                  target_uncond=w.target_uncond, draft_uncond=w.draft_uncond, cfg_scale=w.cfg_scale,
                                  top_k=w.top_k, workspace=ws, stream=stream)
            keep.append((w, out, ws, prm))

        def enqueue(i):
            csd.csd_verify_similar(keep[i % ring_n][3], table, 2.0)
    else:
        from paper_2601_09212_b200.vocab_sharded import ShardedRound, csd_verify_sharded
        n_sh = 4 if kind == "sharded4" else 1
        Vs = V // n_sh
        sched = csd.csd_make_schedule(1, 1.1, 0.7, L)
        step_bytes = 2 * arrays * L * Vs * es * B
        units, unit_name = B * L, "verified_draft_tokens_per_sec"
        op = f"csd_shard_stats/partial/pick/emit on one rank's slice of {Vs} of {V} tokens ({n_sh} slices; gathers are views)"
        ring_n = max(2, -(-2 * L2_BYTES // step_bytes))
        skw = {k: v for k, v in kw.items() if k != "top_k"}   # (top-k is not part of the sharded round)
        for s_ in range(ring_n):
            w = W.make(name, seed=1, step=s_, schedule=sched, device=dev, **skw)
            cut = lambda t: None if t is None else t[:, :, :Vs].contiguous()
            rd = ShardedRound(cut(w.target_logits), cut(w.draft_logits), w.draft_tokens, w.uniforms, w.relax_schedule,
                              v_offset=0, V_total=V, shard=0, n_shards=n_sh, target_uncond=cut(w.target_uncond),
                              draft_uncond=cut(w.draft_uncond), cfg_scale=w.cfg_scale, stream=stream)
            out = (torch.empty(B, L + 1, dtype=torch.int32, device=dev), torch.empty(B, dtype=torch.int32, device=dev))
            keep.append((w, rd, out))
        # every "rank" of the stand-in gather holds this rank's buffer: shapes and kernels are those of n_sh ranks
        gather = lambda t: t.unsqueeze(0).expand((n_sh,) + tuple(t.shape)).contiguous() if n_sh > 1 else t.unsqueeze(0)

        def enqueue(i):
            _, rd, out = keep[i % ring_n]
            csd_verify_sharded(rd, out[0], out[1], gather=gather)

    graph_steps = ring_n * max(1, -(-32 // ring_n))
    with torch.cuda.stream(stream):
        for i in range(ring_n):
            enqueue(i)
    stream.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=stream):
        for i in range(graph_steps):
            enqueue(i)
    replays = max(1, min(args.steps, 512) // graph_steps)
    with torch.cuda.stream(stream):
        graph.replay()
    stream.synchronize()
    reps = []
    for _ in range(5):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            e0.record(stream)
            for _r in range(replays):
                graph.replay()
            e1.record(stream)
        stream.synchronize()
        reps.append(e0.elapsed_time(e1))
    reps.sort()
    steps = replays * graph_steps
    ms = reps[len(reps) // 2]
    peak, peak_kind = measured_peak()
    achieved = step_bytes / (ms * 1e-3 / steps) / 1e9
    print(json.dumps({
        "metric": unit_name, "value": units * steps / (ms * 1e-3), "unit": "1/s", "n_gpus": 1,
        "steps": steps, "reps": len(reps), "ms_per_step": ms / steps, "higher_is_better": True, "data": "synthetic",
        "config": dict(describe(name, kw, "exp delta=1.1 nu=0.7"), op=op,
                       launch=f"CUDA graph of {graph_steps} calls in stream order, {replays} replays, median of {len(reps)}"),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": peak_kind, "bytes_per_launch": step_bytes, "traffic": None},
    }))


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--monitors", action="store_true",
                    help="also ask for the per-position monitors of Theorem 2 (a second pass over every row)")
    ap.add_argument("--single-call-latency", action="store_true",
                    help="csd_params.back_to_back = 0: ordinary stream order, each call spread over the whole GPU")
    ap.add_argument("--steps", type=int, default=2048)
    ap.add_argument("--warmup", type=int, default=64)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="C3")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--drafting-stage", action="store_true",
                    help="side measurement: time csd_sample_rows on the workload's drafter rows instead of the round")
    ap.add_argument("--widened", default=None, choices=["tree", "similar", "sharded", "sharded4"],
                    help="side measurement of a widened entry point on the workload's shapes (see run_widened)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.widened:
        run_widened(args)
    elif args.drafting_stage:
        run_drafting_stage(args)
    else:
        run_native(args)


if __name__ == "__main__":
    main()

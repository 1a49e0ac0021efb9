#!/usr/bin/env python
"""Throughput of the verify-and-feedback step on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg5] [--impl ours|reference]

One step = one pass of the whole hot path (softmax statistics, rejection tests, residual / bonus
draw, KL loss and its gradient) over one batch.  Prints ONE JSON line (rank 0).

  value      verified draft positions per second, inputs resident in HBM, timed with CUDA events
             on the launching stream over exactly K steps, max over ranks
  roofline   algorithmic bytes (read (2k+1)*V*B logits, write k*V*B gradient entries) per launch
             over the mean kernel duration, against the measured HBM copy bandwidth
  e2e        the same metric through the host-memory entry point: pinned host buffers in, host
             buffers out, every copy inside the timed region
  cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload
  --impl reference  times the CPU oracle on the host cores (there is no other implementation of
             this path to run); rank 0 only

With N > 1 (launched by torch.distributed.run) every rank runs the full batch of its own
(weak scaling: sequences are independent, no collective on the path).

  --path greedy   times greedy verification instead (Algorithm 1 in the limit tau -> 0, the decoding
             mode of the paper's experiments): only the target logits are read, (k+1)*V*B entries per
             launch; the line has the same keys, with "path": "greedy" in config.  Not the headline.
  --path ensemble  times the feedback of an online ensemble of --learners N draft models (Sec. 3.3):
             (k + N*k)*V*B logits in, N*k*V*B gradient entries out per launch; value counts the B*k
             positions of the round (each served for all N learners).  Not the headline.
  --path errors   times the step with the feedback restricted to the error position (what OSD
             collects, Sec. 3.1): (2k+1)*V*B logits in, B*V gradient entries out.  Not the headline.
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

from paper_2603_12617_b200 import synth  # noqa: E402

METRIC = "verified draft positions/sec"
UNIT = "positions/s"
L2_BYTES = 126 * 1024 * 1024
# dram__bytes_read.sum + dram__bytes_write.sum per launch at full size, from the ncu captures
# summarised under profiles/ (bytes; a workload that is not listed has not been captured)
NCU_TRAFFIC_ENSEMBLE = {("cfg5", 3): 3388811776 + 2325275904}
NCU_TRAFFIC_ERRORS = {"cfg5": 1707537664 + 3327232 + 251808256 + 99995904}   # both kernels of the step
NCU_TRAFFIC_GREEDY = {"cfg5": 919481088 + 244224}
NCU_TRAFFIC_BYTES = {"cfg5": 2078492160 + 758877952, "cfg3": 155482368 + 36729856, "cfg4": 179505152 + 50643456}


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return 6650.0, "fallback (6.65 TB/s, earlier measurement on this pool)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if hasattr(uuid, "encode") else uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception as exc:  # NVML missing: report that, do not fail the run
            self._nv, self._err = None, repr(exc)

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for bit, name in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.004)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if self._nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable: " + self._err]}
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def time_oracle(inp, seqs, nthreads):
    from oracle import sd_oracle
    sl = np.asarray(seqs)
    t0 = time.perf_counter()
    sd_oracle.verify_feedback(inp.target_logits[sl], inp.draft_logits[sl], inp.draft_tokens[sl],
                              inp.uniforms[sl], inp.tau, nthreads=nthreads)
    return time.perf_counter() - t0


def cpu_baseline(cfg, inp, target_seconds=12.0):
    """The oracle on the host cores over a bounded sample of the workload's sequences."""
    from oracle import sd_oracle
    cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
    n = min(cfg.B, cores)
    t = time_oracle(inp, range(n), cores)
    if t < target_seconds / 2 and n < cfg.B:
        n2 = int(min(cfg.B, max(n, n * target_seconds / max(t, 1e-3))))
        n2 = max(cores, n2 // cores * cores)
        if n2 > n:
            n, t = n2, time_oracle(inp, range(n2), cores)
    return {"value": n * cfg.k / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} of {cfg.B} sequences of {cfg.name} (k={cfg.k}, V={cfg.V}, {cfg.dtype}), "
                      f"one call, {t:.2f} s",
            "gb_per_s": n * cfg.algorithmic_bytes / cfg.B / t / 1e9}


def run_reference(args, cfg):
    """--impl reference: the CPU oracle timed on the host cores, bounded sample per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import sd_oracle
    sd_oracle.build()
    cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
    # a step is the oracle on n sequences; n is sized so the run ends within about two minutes
    probe_cfg = cfg.with_batch(min(cfg.B, cores))
    inp = synth.make_inputs(probe_cfg)
    t_probe = time_oracle(inp, range(probe_cfg.B), cores)
    budget = 120.0 / max(1, args.steps + args.warmup)
    n = probe_cfg.B
    if t_probe > budget:
        n = max(1, int(probe_cfg.B * budget / t_probe))
    threads = min(cores, n)
    for _ in range(args.warmup):
        time_oracle(inp, range(n), threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        time_oracle(inp, range(n), threads)
    dt = time.perf_counter() - t0
    value = args.steps * n * cfg.k / dt
    sample = f"{n} of {cfg.B} sequences of {cfg.name} per step, {threads} threads"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype + " inputs, f64 arithmetic",
            "data": "synthetic", "config": workload_config(cfg, note="CPU oracle on a bounded sample per step"),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(cfg, **extra):
    d = {"workload": f"{cfg.name}: B={cfg.B}, k={cfg.k}, V={cfg.V}, {cfg.dtype} logits, tau={cfg.tau}, "
                     f"recipe={cfg.recipe}", "B": cfg.B, "k": cfg.k, "V": cfg.V, "logits": cfg.dtype,
         "temperature": cfg.tau}
    d.update(extra)
    return d


def run_ours(args, cfg):
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding, shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        if world == 1 and args.gpus > 1:
            raise SystemExit("launch with torch.distributed.run for --gpus > 1")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    # every rank verifies a full batch of its own (different seed per rank): weak scaling
    inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16

    def as_torch(a):
        t = torch.from_numpy(a)
        return t.view(torch.bfloat16) if a.dtype == np.uint16 else t

    hT, hD = as_torch(inp.target_logits).pin_memory(), as_torch(inp.draft_logits).pin_memory()
    hx, hu = torch.from_numpy(inp.draft_tokens).pin_memory(), torch.from_numpy(inp.uniforms).pin_memory()
    in_bytes = hT.numel() * hT.element_size() + hD.numel() * hD.element_size()
    # inputs larger than L2, or enough rotating copies that every step reads from HBM
    nsets = 1 if in_bytes > 2 * L2_BYTES else int(min(64, -(-3 * L2_BYTES // in_bytes)))
    sets = []
    for _ in range(nsets):
        sets.append((hT.to(dev), hD.to(dev), hx.to(dev), hu.to(dev)))
    out = binding.StepOutputs(
        accept_len=torch.empty(cfg.B, dtype=torch.int32, device=dev),
        tokens=torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32, device=dev),
        loss=torch.empty((cfg.B, cfg.k), dtype=torch.float32, device=dev),
        grad_draft=torch.empty((cfg.B, cfg.k, cfg.V), dtype=tdt, device=dev))

    def step(i):
        T, D, x, u = sets[i % nsets]
        binding.sd_verify_feedback(T, D, x, u, inp.tau, out=out)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    info = binding.sd_launch_info()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        t_begin.record()
        for i in range(args.steps):
            starts[i].record()
            step(i)
            ends[i].record()
        t_end.record()
        barrier()
    total_ms = shard.max_over_ranks(t_begin.elapsed_time(t_end), device=str(dev) if world > 1 else "cpu")
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    mean_kernel_ms = float(np.mean(kernel_ms))
    if args.times_out and rank == 0:
        with open(args.times_out, "w") as fh:
            json.dump(kernel_ms, fh)
    positions = cfg.B * cfg.k * world
    value = positions * args.steps / (total_ms * 1e-3)

    # sanity: the timed outputs are the real ones (checked against the oracle on a few sequences)
    check_seqs = [0, cfg.B // 2, cfg.B - 1] if cfg.B > 2 else list(range(cfg.B))
    verified = None
    if rank == 0:
        from oracle import sd_oracle
        sl = np.asarray(sorted(set(check_seqs)))
        ref = sd_oracle.verify_feedback(inp.target_logits[sl], inp.draft_logits[sl], inp.draft_tokens[sl],
                                        inp.uniforms[sl], inp.tau, want_grad=False, nthreads=len(sl))
        T, D, x, u = sets[0]
        chk = binding.sd_verify_feedback(T, D, x, u, inp.tau)
        torch.cuda.synchronize()
        safe = (ref.accept_band.sum(1) == 0) & (ref.cdf_margin > 1e-6)
        verified = bool((chk.accept_len.cpu().numpy()[sl][safe] == ref.accept_len[safe]).all()
                        and (chk.tokens.cpu().numpy()[sl][safe] == ref.tokens[safe]).all()
                        and np.allclose(chk.loss.cpu().numpy()[sl], ref.loss, rtol=2e-2 if cfg.dtype == "bf16" else 1e-5, atol=4e-7))

    # end to end through the host-memory entry point: pinned host buffers, copies inside the region
    e2e_steps = max(1, min(args.steps, 10))
    hout = binding.StepOutputs(
        accept_len=torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
        tokens=torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory(),
        loss=torch.empty((cfg.B, cfg.k), dtype=torch.float32).pin_memory(),
        grad_draft=torch.empty((cfg.B, cfg.k, cfg.V), dtype=tdt).pin_memory())
    for _ in range(2):
        binding.sd_verify_feedback_host(hT, hD, hx, hu, inp.tau, out=hout)
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        binding.sd_verify_feedback_host(hT, hD, hx, hu, inp.tau, out=hout)
    barrier()
    e2e_s = shard.max_over_ranks(time.perf_counter() - t0, device=str(dev) if world > 1 else "cpu")
    h2d = in_bytes + hx.numel() * 4 + hu.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in (hout.accept_len, hout.tokens, hout.loss, hout.grad_draft))
    e2e = {"value": positions * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
           "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "ms_per_step": e2e_s / e2e_steps * 1e3,
           "entry_point": "sd_verify_feedback_host"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_src = measured_peak_gbs()
    achieved = cfg.algorithmic_bytes / (mean_kernel_ms * 1e-3) / 1e9
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "traffic": NCU_TRAFFIC_BYTES.get(cfg.name) if not args.batch else None, "peak_source": peak_src,
                "algorithmic_bytes_per_launch": cfg.algorithmic_bytes, "kernel_ms_mean": mean_kernel_ms,
                "kernel_ms_min": float(np.min(kernel_ms)), "kernel": "sd_stream_kernel" if info["path"] == 1 else "sd_generic_kernel",
                "frac_of_nominal_8000_GBps": achieved / 8000.0}
    # second ceiling: the special-function units (4 ex2 per entry pair and 2 per bonus entry; 16 results per
    # clock and SM, 148 SMs at the maximum SM clock): what binds when entries are 2 bytes
    ex2 = (4 * cfg.k + 2) * cfg.V * cfg.B
    sfu_peak = 148 * 16 * 1.965e9
    roofline["sfu"] = {"ex2_per_launch": ex2, "achieved_per_s": ex2 / (mean_kernel_ms * 1e-3), "peak_per_s": sfu_peak,
                       "frac": ex2 / (mean_kernel_ms * 1e-3) / sfu_peak,
                       "peak_source": "148 SMs x 16 ex2/clk x 1965 MHz (nominal unit count and maximum clock)"}
    base = cpu_baseline(cfg, inp) if not args.no_cpu_baseline else None
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)",
            "data": "synthetic",
            "config": workload_config(cfg, l2="inputs larger than L2" if nsets == 1 else f"{nsets} rotating input sets larger than L2 together",
                                      parallelism=f"replicas x{world}, sequences independent, no collective",
                                      launch=info),
            "roofline": roofline, "cpu_baseline": base, "e2e": e2e, "gpu_launches": args.steps * info["kernels"],
            "clocks": clocks.summary(), "outputs_verified_against_oracle": verified}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_greedy(args, cfg):
    """--path greedy: sd_verify_greedy on the target logits of the workload, one GPU per rank."""
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding, shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
    hT = torch.from_numpy(inp.target_logits)
    if inp.target_logits.dtype == np.uint16:
        hT = hT.view(torch.bfloat16)
    hT = hT.pin_memory()
    # greedy drafting proposes the draft's argmax; the inputs carry sampled tokens, which serves as well:
    # the work does not depend on the tokens
    hx = torch.from_numpy(inp.draft_tokens).pin_memory()
    in_bytes = hT.numel() * hT.element_size()
    nsets = 1 if in_bytes > 2 * L2_BYTES else int(min(64, -(-3 * L2_BYTES // in_bytes)))
    sets = [(hT.to(dev), hx.to(dev)) for _ in range(nsets)]
    out = binding.sd_verify_greedy(*sets[0])

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        binding.sd_verify_greedy(*sets[i % nsets], out=out)
    info = binding.sd_launch_info()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        t_begin.record()
        for i in range(args.steps):
            starts[i].record()
            binding.sd_verify_greedy(*sets[i % nsets], out=out)
            ends[i].record()
        t_end.record()
        barrier()
    total_ms = shard.max_over_ranks(t_begin.elapsed_time(t_end), device=str(dev) if world > 1 else "cpu")
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    mean_kernel_ms = float(np.mean(kernel_ms))
    positions = cfg.B * cfg.k * world
    value = positions * args.steps / (total_ms * 1e-3)

    # end to end: pinned host logits in, results back to the host, every copy inside the region
    e2e_steps = max(1, min(args.steps, 10))
    dT, dx = torch.empty_like(sets[0][0]), torch.empty_like(sets[0][1])
    h_n = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    h_tok = torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory()

    def e2e_step():
        dT.copy_(hT, non_blocking=True)
        dx.copy_(hx, non_blocking=True)
        binding.sd_verify_greedy(dT, dx, out=out)
        h_n.copy_(out.accept_len, non_blocking=True)
        h_tok.copy_(out.tokens, non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = shard.max_over_ranks(time.perf_counter() - t0, device=str(dev) if world > 1 else "cpu")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    from oracle import sd_oracle
    t0 = time.perf_counter()
    ref = sd_oracle.verify_greedy(inp.target_logits, inp.draft_tokens)
    t_cpu = time.perf_counter() - t0
    verified = bool((h_n.numpy() == ref.accept_len).all() and (h_tok.numpy() == ref.tokens).all()
                    and (out.argmax.cpu().numpy() == ref.argmax).all())
    algo = (cfg.k + 1) * cfg.V * cfg.B * cfg.elem_bytes
    peak, peak_src = measured_peak_gbs()
    achieved = algo / (mean_kernel_ms * 1e-3) / 1e9
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32 comparisons" if cfg.dtype == "f32" else "bf16 comparisons",
            "data": "synthetic",
            "config": workload_config(cfg, path="greedy", l2="inputs larger than L2" if nsets == 1 else f"{nsets} rotating input sets larger than L2 together",
                                      parallelism=f"replicas x{world}, sequences independent, no collective", launch=info),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_GREEDY.get(cfg.name) if not args.batch else None,
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": algo,
                         "kernel_ms_mean": mean_kernel_ms, "kernel_ms_min": float(np.min(kernel_ms)),
                         "kernel": "sd_greedy_kernel"},
            "cpu_baseline": {"value": cfg.B * cfg.k / t_cpu, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"all {cfg.B} sequences of {cfg.name}, one call, {t_cpu:.2f} s"},
            "e2e": {"value": positions * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(in_bytes + hx.numel() * 4),
                    "d2h_bytes_per_step": int(h_n.numel() * 4 + h_tok.numel() * 4), "steps": e2e_steps,
                    "ms_per_step": e2e_s / e2e_steps * 1e3, "entry_point": "sd_verify_greedy between pinned-memory copies"},
            "gpu_launches": args.steps * info["kernels"], "clocks": clocks.summary(),
            "outputs_verified_against_oracle": verified}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_errors(args, cfg):
    """--path errors: sd_verify_error_feedback on the workload, one GPU per rank."""
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding, shard

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)

    def as_torch(a):
        t = torch.from_numpy(a)
        return t.view(torch.bfloat16) if a.dtype == np.uint16 else t

    hT, hD = as_torch(inp.target_logits).pin_memory(), as_torch(inp.draft_logits).pin_memory()
    hx, hu = torch.from_numpy(inp.draft_tokens).pin_memory(), torch.from_numpy(inp.uniforms).pin_memory()
    in_bytes = hT.numel() * hT.element_size() + hD.numel() * hD.element_size()
    nsets = 1 if in_bytes > 2 * L2_BYTES else int(min(64, -(-3 * L2_BYTES // in_bytes)))
    sets = [(hT.to(dev), hD.to(dev), hx.to(dev), hu.to(dev)) for _ in range(nsets)]
    out = binding.sd_verify_error_feedback(*sets[0], inp.tau)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        binding.sd_verify_error_feedback(*sets[i % nsets], inp.tau, out=out)
    info = binding.sd_launch_info()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        t_begin.record()
        for i in range(args.steps):
            starts[i].record()
            binding.sd_verify_error_feedback(*sets[i % nsets], inp.tau, out=out)
            ends[i].record()
        t_end.record()
        barrier()
    total_ms = shard.max_over_ranks(t_begin.elapsed_time(t_end), device=str(dev) if world > 1 else "cpu")
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    mean_kernel_ms = float(np.mean(kernel_ms))
    positions = cfg.B * cfg.k * world
    value = positions * args.steps / (total_ms * 1e-3)

    # end to end: pinned host logits in, results and the gradient rows back to the host
    e2e_steps = max(1, min(args.steps, 10))
    dbuf = [torch.empty_like(t) for t in sets[0]]
    h_n = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
    h_tok = torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory()
    h_loss = torch.empty((cfg.B, cfg.k), dtype=torch.float32).pin_memory()
    h_g = torch.empty((cfg.B, cfg.V), dtype=hT.dtype).pin_memory()

    def e2e_step():
        for a, b in zip(dbuf, (hT, hD, hx, hu)):
            a.copy_(b, non_blocking=True)
        binding.sd_verify_error_feedback(*dbuf, inp.tau, out=out)
        h_n.copy_(out.accept_len, non_blocking=True)
        h_tok.copy_(out.tokens, non_blocking=True)
        h_loss.copy_(out.loss, non_blocking=True)
        h_g.copy_(out.error_grad, non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = shard.max_over_ranks(time.perf_counter() - t0, device=str(dev) if world > 1 else "cpu")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    from oracle import sd_oracle
    cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
    nseq = min(cfg.B, cores)
    sl = np.arange(nseq)
    t0 = time.perf_counter()
    ref = sd_oracle.error_position_feedback(inp.target_logits[sl], inp.draft_logits[sl], inp.draft_tokens[sl],
                                            inp.uniforms[sl], inp.tau, nthreads=cores)
    t_cpu = time.perf_counter() - t0
    safe = (ref.full.accept_band.sum(1) == 0) & (ref.full.cdf_margin > 1e-6)
    g = h_g[:nseq].float().numpy().astype(np.float64)
    tol = 2e-2 if cfg.dtype == "bf16" else 1e-5
    verified = bool((h_n.numpy()[sl][safe] == ref.full.accept_len[safe]).all()
                    and (h_tok.numpy()[sl][safe] == ref.full.tokens[safe]).all()
                    and np.allclose(h_loss.numpy()[sl], ref.full.loss, rtol=tol, atol=4e-7)
                    and all(np.abs(g[b] - ref.error_grad[b]).max() <= tol * np.abs(ref.error_grad[b]).max() + 1e-6
                            for b in range(nseq) if safe[b]))
    s = cfg.elem_bytes
    algo = ((2 * cfg.k + 1) + 1) * cfg.V * cfg.B * s
    peak, peak_src = measured_peak_gbs()
    achieved = algo / (mean_kernel_ms * 1e-3) / 1e9
    d2h = h_n.numel() * 4 + h_tok.numel() * 4 + h_loss.numel() * 4 + h_g.numel() * h_g.element_size()
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)",
            "data": "synthetic",
            "config": workload_config(cfg, path="errors", mean_accept_len=float(h_n.float().mean()),
                                      l2="inputs larger than L2" if nsets == 1 else f"{nsets} rotating input sets larger than L2 together",
                                      parallelism=f"replicas x{world}, sequences independent, no collective", launch=info),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_ERRORS.get(cfg.name) if not args.batch else None,
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": algo,
                         "kernel_ms_mean": mean_kernel_ms, "kernel_ms_min": float(np.min(kernel_ms)),
                         "kernel": "sd_stream_kernel<pass 1 only> + sd_errpos_kernel"},
            "cpu_baseline": {"value": nseq * cfg.k / t_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{nseq} of {cfg.B} sequences of {cfg.name}, one call, {t_cpu:.2f} s"},
            "e2e": {"value": positions * e2e_steps / e2e_s, "unit": UNIT,
                    "h2d_bytes_per_step": int(in_bytes + hx.numel() * 4 + hu.numel() * 4), "d2h_bytes_per_step": int(d2h),
                    "steps": e2e_steps, "ms_per_step": e2e_s / e2e_steps * 1e3,
                    "entry_point": "sd_verify_error_feedback between pinned-memory copies"},
            "gpu_launches": args.steps * info["kernels"], "clocks": clocks.summary(),
            "outputs_verified_against_oracle": verified}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_ensemble(args, cfg):
    """--path ensemble: sd_ensemble_feedback with N learners on the workload, one GPU per rank."""
    import torch
    import torch.distributed as dist

    import __graft_entry__ as entry
    entry.build()
    from paper_2603_12617_b200 import binding, shard

    N = args.learners
    eps = 10.0
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
    drafts = synth.ensemble_drafts(inp, N, seed=synth.BASE_SEED + 1000 * rank)

    def as_torch(a):
        t = torch.from_numpy(a)
        return t.view(torch.bfloat16) if a.dtype == np.uint16 else t

    hT = as_torch(inp.target_logits).pin_memory()
    hD = [as_torch(d).pin_memory() for d in drafts]
    in_bytes = hT.numel() * hT.element_size() + sum(d.numel() * d.element_size() for d in hD)
    nsets = 1 if in_bytes > 2 * L2_BYTES else int(min(64, -(-3 * L2_BYTES // in_bytes)))
    sets = [(hT.to(dev), [d.to(dev) for d in hD]) for _ in range(nsets)]
    out = binding.sd_ensemble_feedback(sets[0][0], sets[0][1], inp.tau, eps)
    cum = torch.zeros(N, dtype=torch.float64, device=dev)

    def step(i):
        T, Ds = sets[i % nsets]
        binding.sd_ensemble_feedback(T, Ds, inp.tau, eps, cum_loss=cum, out=out)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(max(3, args.warmup)):
        step(i)
    info = binding.sd_launch_info()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local) as clocks:
        t_begin.record()
        for i in range(args.steps):
            starts[i].record()
            step(i)
            ends[i].record()
        t_end.record()
        barrier()
    total_ms = shard.max_over_ranks(t_begin.elapsed_time(t_end), device=str(dev) if world > 1 else "cpu")
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    mean_kernel_ms = float(np.mean(kernel_ms))
    positions = cfg.B * cfg.k * world
    value = positions * args.steps / (total_ms * 1e-3)

    # end to end: pinned host logits in, losses, weights and gradients back to the host
    e2e_steps = max(1, min(args.steps, 5))
    dT, dD = torch.empty_like(sets[0][0]), [torch.empty_like(d) for d in sets[0][1]]
    h_loss = torch.empty((N, cfg.B, cfg.k), dtype=torch.float32).pin_memory()
    h_w = torch.empty(N, dtype=torch.float32).pin_memory()
    h_grad = [torch.empty_like(d).pin_memory() for d in hD]

    def e2e_step():
        dT.copy_(hT, non_blocking=True)
        for a, b in zip(dD, hD):
            a.copy_(b, non_blocking=True)
        binding.sd_ensemble_feedback(dT, dD, inp.tau, eps, cum_loss=cum, out=out)
        h_loss.copy_(out.loss, non_blocking=True)
        h_w.copy_(out.weights, non_blocking=True)
        for a, b in zip(h_grad, out.grad):
            a.copy_(b, non_blocking=True)
        torch.cuda.synchronize()

    e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        e2e_step()
    barrier()
    e2e_s = shard.max_over_ranks(time.perf_counter() - t0, device=str(dev) if world > 1 else "cpu")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # the timed outputs against the oracle on a few sequences, and the oracle's own speed
    from oracle import sd_oracle
    cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
    nseq = min(cfg.B, max(1, cores // cfg.k))
    sl = np.arange(nseq)
    t0 = time.perf_counter()
    ref = sd_oracle.ensemble_feedback(inp.target_logits[sl], [d[sl] for d in drafts], inp.tau, eps, want_grad=False,
                                      nthreads=cores)
    t_cpu = time.perf_counter() - t0
    loss = h_loss.numpy()[:, :nseq].astype(np.float64)
    verified = bool(np.allclose(loss, ref.loss, rtol=2e-2 if cfg.dtype == "bf16" else 1e-5, atol=4e-7)
                    and abs(float(h_w.sum()) - 1.0) < 1e-5)
    s = cfg.elem_bytes
    algo = ((cfg.k + N * cfg.k) + N * cfg.k) * cfg.V * cfg.B * s
    d2h = h_loss.numel() * 4 + h_w.numel() * 4 + sum(g.numel() * g.element_size() for g in h_grad)
    peak, peak_src = measured_peak_gbs()
    achieved = algo / (mean_kernel_ms * 1e-3) / 1e9
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)",
            "data": "synthetic",
            "config": workload_config(cfg, path="ensemble", learners=N, epsilon=eps,
                                      l2="inputs larger than L2" if nsets == 1 else f"{nsets} rotating input sets larger than L2 together",
                                      parallelism=f"replicas x{world}, sequences independent, no collective", launch=info),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         "traffic": NCU_TRAFFIC_ENSEMBLE.get((cfg.name, N)) if not args.batch else None,
                         "peak_source": peak_src, "algorithmic_bytes_per_launch": algo,
                         "kernel_ms_mean": mean_kernel_ms, "kernel_ms_min": float(np.min(kernel_ms)),
                         "kernel": "sd_stream_kernel<ensemble> + sd_hedge_kernel"},
            "cpu_baseline": {"value": nseq * cfg.k / t_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                             "sample": f"{nseq} of {cfg.B} sequences of {cfg.name}, {N} learners, no gradients, "
                                       f"one call, {t_cpu:.2f} s"},
            "e2e": {"value": positions * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(in_bytes),
                    "d2h_bytes_per_step": int(d2h), "steps": e2e_steps, "ms_per_step": e2e_s / e2e_steps * 1e3,
                    "entry_point": "sd_ensemble_feedback between pinned-memory copies"},
            "gpu_launches": args.steps * info["kernels"], "clocks": clocks.summary(),
            "outputs_verified_against_oracle": verified}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default="cfg5", choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=0, help="override B (profiling on a smaller case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--path", choices=["sample", "greedy", "ensemble", "errors"], default="sample",
                    help="sample: the verify-and-feedback step (the headline); greedy: greedy verification; "
                         "ensemble: feedback of an online ensemble of draft models; errors: feedback at the error position only")
    ap.add_argument("--learners", type=int, default=3, help="draft models of --path ensemble")
    ap.add_argument("--times-out", default="", help="write the per-step device times (ms) of the headline path here")
    args = ap.parse_args()
    cfg = synth.CONFIGS[args.config]
    if args.batch:
        cfg = cfg.with_batch(args.batch)
    if args.impl == "reference":
        run_reference(args, cfg)
    elif args.path == "greedy":
        run_greedy(args, cfg)
    elif args.path == "ensemble":
        run_ensemble(args, cfg)
    elif args.path == "errors":
        run_errors(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()

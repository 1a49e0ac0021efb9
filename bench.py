#!/usr/bin/env python
"""Throughput of the verify-and-feedback step on synthetic workloads.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config cfg5] [--impl ours|reference]

One step = one pass of the whole hot path (softmax statistics, rejection tests, residual / bonus
draw, KL loss and its gradient) over one batch.  Prints ONE JSON line (rank 0).

  value      verified draft positions per second, inputs resident in HBM, timed with CUDA events
             on the launching stream over exactly K steps, max over ranks
  roofline   algorithmic bytes (read (2k+1)*V*B logits, write k*V*B gradient entries) per launch
             over the mean kernel duration, against the measured HBM copy bandwidth
  e2e        the same metric through host buffers: pinned host memory in, host buffers out, every
             copy inside the timed region (the headline path: sd_verify_feedback_host)
  cpu_baseline  the CPU oracle, as it stands, on a bounded sample of the same workload
  parity     the timed outputs against the oracle on that sample: sequences compared, rows inside the
             two threshold bands, mismatches inside and outside them, mean accept length, mean sum min(p,q)
  --impl reference  times the CPU oracle on the host cores (there is no other implementation of
             this path to run); rank 0 only

With N > 1 every rank runs the full batch of its own (weak scaling: sequences are independent, no
collective on the path).  Started without torch.distributed.run, `--gpus N` starts its own ranks.

  --path greedy    greedy verification (Algorithm 1 in the limit tau -> 0): (k+1)*V*B entries read
  --path ensemble  feedback of an online ensemble of --learners N draft models (Sec. 3.3)
  --path errors    feedback restricted to the error position (what OSD collects, Sec. 3.1)
  --path lmhead    the step after the path: the output layer's gradient dW = g^T X on the tensor cores,
                   R = B*k positions of the workload, --features d; roofline in TFLOP/s
Each prints the same keys with "path" in config; none of them is the headline.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import socket
import subprocess
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
TOL = {"f32": 1e-5, "bf16": 2e-2}


def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as fh:
            d = json.load(fh)
        return {"hbm_gbs": float(d["hbm_gbs"]), "bf16_tflops": float(d["bf16_tflops"]),
                "bf16_tflops_sustained": float(d["bf16_tflops_sustained"]), "source": "measured (MEASURED_PEAKS.json)"}
    except Exception:
        return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0,
                "source": "fallback (6.65 TB/s, 1.59 PFLOP/s burst, 1.4 sustained)"}


def kernel_source_hash() -> str:
    """Identifies the kernels a DRAM-traffic capture belongs to: the CUDA sources without their
    comments and blank space, hashed (a reworded comment does not change a kernel)."""
    import re
    h = hashlib.sha256()
    src = os.path.join(ROOT, "paper_2603_12617_b200", "csrc")
    for name in sorted(os.listdir(src)):
        with open(os.path.join(src, name), "r", encoding="utf-8") as fh:
            text = fh.read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        text = re.sub(r"//[^\n]*", "", text)
        h.update(name.encode())
        h.update("".join(text.split()).encode())
    return h.hexdigest()[:16]


def captured_traffic(path: str, cfg_name: str, extra: str = "-"):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch from the ncu capture summarised in
    profiles/dram_traffic.txt -- only if the kernels have not changed since it was taken."""
    fname = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    try:
        with open(fname) as fh:
            rows = [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]
    except OSError:
        return None, "no capture on file"
    for row in rows:
        if len(row) >= 6 and row[0] == path and row[1] == cfg_name and row[2] == extra:
            if row[5] != kernel_source_hash():
                return None, "the kernels have changed since the capture in profiles/dram_traffic.txt"
            return int(row[3]) + int(row[4]), "ncu capture summarised in profiles/dram_traffic.txt (same kernel sources)"
    return None, "this workload has not been captured"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int):
        self.samples, self.reasons = [], set()
        self.mem_samples, self.power_samples = [], []
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

    def _sample(self):
        nv = self._nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
            self.mem_samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_MEM)))
            self.power_samples.append(nv.nvmlDeviceGetPowerUsage(self._h) / 1000.0)
            mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
            for bit, name in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self._sample()
            time.sleep(0.004)

    def __enter__(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def sample_now(self):
        """One more sample from the calling thread (the GPU is still under load when this is called)."""
        if self._nv is not None:
            self._sample()

    def __exit__(self, *a):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if self._nv is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvml unavailable: " + self._err]}
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples),
                "sm_mhz_min": float(min(self.samples)) if self.samples else None,
                "mem_mhz": float(np.median(self.mem_samples)) if self.mem_samples else None,
                "mem_mhz_min": float(min(self.mem_samples)) if self.mem_samples else None,
                "power_w_max": float(max(self.power_samples)) if self.power_samples else None}


# ------------------------------------------------------------------------------------------
# the oracle legs

def run_oracle(inp, seqs, nthreads, want_grad=True):
    from oracle import sd_oracle
    sl = np.asarray(seqs)
    t0 = time.perf_counter()
    res = sd_oracle.verify_feedback(inp.target_logits[sl], inp.draft_logits[sl], inp.draft_tokens[sl],
                                    inp.uniforms[sl], inp.tau, want_grad=want_grad, nthreads=nthreads)
    return time.perf_counter() - t0, res


def cpu_baseline(cfg, inp, target_seconds=12.0):
    """The oracle on the host cores over a bounded sample of the workload's sequences; also returns
    the sequences and the oracle's result for them (the parity counts of the line come from it)."""
    from oracle import sd_oracle
    cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
    n = min(cfg.B, cores)
    t, res = run_oracle(inp, range(n), cores)
    if t < target_seconds / 2 and n < cfg.B:
        n2 = int(min(cfg.B, max(n, n * target_seconds / max(t, 1e-3))))
        n2 = max(cores, n2 // cores * cores)
        if n2 > n:
            n = n2
            t, res = run_oracle(inp, range(n2), cores)
    base = {"value": n * cfg.k / t, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"{n} of {cfg.B} sequences of {cfg.name} (k={cfg.k}, V={cfg.V}, {cfg.dtype}), "
                      f"one call, {t:.2f} s",
            "gb_per_s": n * cfg.algorithmic_bytes / cfg.B / t / 1e9}
    return base, np.arange(n), res


def parity_counts(cfg, ref, seqs, accept_len, tokens, loss):
    """The timed outputs against the oracle on `seqs`: rows in the two threshold bands, mismatches
    inside and outside them, and whether the losses hold the tolerance."""
    n_gpu, tok_gpu = accept_len[seqs], tokens[seqs]
    accept_band = ref.accept_band.sum(1) > 0
    sample_band = ref.cdf_margin <= 1e-6
    band = accept_band | sample_band
    mismatch = (n_gpu != ref.accept_len) | (tok_gpu != ref.tokens).any(axis=1)
    out = {"sequences_compared": int(len(seqs)), "accept_band_rows": int(ref.accept_band.sum()),
           "sample_band_rows": int(sample_band.sum()), "mismatches_inside_the_bands": int((mismatch & band).sum()),
           "mismatches_outside_the_bands": int((mismatch & ~band).sum()),
           "mean_accept_len": float(accept_len.mean()), "mean_acc_prob_oracle": float(ref.acc_prob.mean())}
    if loss is not None:
        err = np.abs(loss[seqs].astype(np.float64) - ref.loss)
        out["loss_within_tolerance"] = bool((err <= TOL[cfg.dtype] * np.maximum(np.abs(ref.loss), 1e-6)).all())
    return out


def run_reference(args, cfg):
    """--impl reference: the CPU oracle timed on the host cores, bounded sample per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from oracle import sd_oracle
    sd_oracle.build()
    cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
    # a step is the oracle on n sequences; n is sized so the run ends within about two minutes
    probe_cfg = cfg.with_batch(min(cfg.B, cores))
    inp = synth.make_inputs(probe_cfg)
    t_probe, _ = run_oracle(inp, range(probe_cfg.B), cores)
    budget = 120.0 / max(1, args.steps + args.warmup)
    n = probe_cfg.B
    if t_probe > budget:
        n = max(1, int(probe_cfg.B * budget / t_probe))
    threads = min(cores, n)
    for _ in range(args.warmup):
        run_oracle(inp, range(n), threads)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run_oracle(inp, range(n), threads)
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


# ------------------------------------------------------------------------------------------
# the paths: each describes one entry point to the common timing loop

def as_torch(a):
    import torch
    t = torch.from_numpy(a)
    return t.view(torch.bfloat16) if a.dtype == np.uint16 else t


def rotating_sets(host_tensors, dev):
    """Device copies of the inputs: one set if it is larger than L2 by itself, else enough rotating
    sets that every step reads from HBM."""
    in_bytes = sum(t.numel() * t.element_size() for t in host_tensors)
    nsets = 1 if in_bytes > 2 * L2_BYTES else int(min(64, -(-3 * L2_BYTES // in_bytes)))
    return [[t.to(dev) for t in host_tensors] for _ in range(nsets)], in_bytes, nsets


class SamplePath:
    """The headline: sd_verify_feedback (library scratch), e2e through sd_verify_feedback_host."""
    name, kernel, traffic_path = "sample", "sd_stream_kernel", "sample"

    def __init__(self, args, cfg, dev, rank, binding):
        import torch
        self.b, self.cfg, self.torch = binding, cfg, torch
        self.inp = inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
        self.host = [as_torch(inp.target_logits).pin_memory(), as_torch(inp.draft_logits).pin_memory(),
                     torch.from_numpy(inp.draft_tokens).pin_memory(), torch.from_numpy(inp.uniforms).pin_memory()]
        self.sets, self.in_bytes, self.nsets = rotating_sets(self.host, dev)
        tdt = self.host[0].dtype
        self.out = binding.StepOutputs(
            accept_len=torch.empty(cfg.B, dtype=torch.int32, device=dev),
            tokens=torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32, device=dev),
            loss=torch.empty((cfg.B, cfg.k), dtype=torch.float32, device=dev),
            grad_draft=torch.empty((cfg.B, cfg.k, cfg.V), dtype=tdt, device=dev))
        self.algorithmic = cfg.algorithmic_bytes
        self.positions = cfg.B * cfg.k
        self.dtype = "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)"
        self.extra = {}
        self.e2e_entry = "sd_verify_feedback_host"

    def step(self, i):
        T, D, x, u = self.sets[i % self.nsets]
        self.b.sd_verify_feedback(T, D, x, u, self.inp.tau, out=self.out)

    def e2e_prepare(self):
        torch, cfg = self.torch, self.cfg
        self.hout = self.b.StepOutputs(
            accept_len=torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
            tokens=torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory(),
            loss=torch.empty((cfg.B, cfg.k), dtype=torch.float32).pin_memory(),
            grad_draft=torch.empty((cfg.B, cfg.k, cfg.V), dtype=self.host[0].dtype).pin_memory())
        self.h2d = self.in_bytes
        self.d2h = sum(t.numel() * t.element_size() for t in (self.hout.accept_len, self.hout.tokens, self.hout.loss, self.hout.grad_draft))

    def e2e_step(self):
        self.b.sd_verify_feedback_host(*self.host, self.inp.tau, out=self.hout)

    def finish(self, args):
        """CPU baseline and parity of the timed outputs (rank 0)."""
        torch, cfg = self.torch, self.cfg
        T, D, x, u = self.sets[0]
        chk = self.b.sd_verify_feedback(T, D, x, u, self.inp.tau)
        torch.cuda.synchronize()
        if args.no_cpu_baseline:
            seqs = np.asarray(sorted({0, cfg.B // 2, cfg.B - 1}))
            base, (_, ref) = None, run_oracle(self.inp, seqs, len(seqs), want_grad=False)
        else:
            base, seqs, ref = cpu_baseline(cfg, self.inp)
        parity = parity_counts(cfg, ref, seqs, chk.accept_len.cpu().numpy(), chk.tokens.cpu().numpy(), chk.loss.cpu().numpy())
        verified = parity["mismatches_outside_the_bands"] == 0 and parity.get("loss_within_tolerance", True)
        return base, parity, bool(verified)


class HintPath(SamplePath):
    """sd_verify_feedback_hint: the step plus the hint error of the optimistic update, the gradient
    written over the hint in place.  One more read of B*k*V entries per step than the headline."""
    name, kernel, traffic_path = "hint", "sd_stream_kernel", "hint"

    def __init__(self, args, cfg, dev, rank, binding):
        super().__init__(args, cfg, dev, rank, binding)
        torch = self.torch
        code = binding.SD_DTYPE_F32 if cfg.dtype == "f32" else binding.SD_DTYPE_BF16
        self.ws = torch.empty(binding.sd_hint_workspace_bytes(cfg.B, cfg.k, cfg.V, code), dtype=torch.uint8, device=dev)
        # the buffer that holds the last round's gradient on entry and this round's on return
        self.hint = self.out.grad_draft
        self.hint.zero_()
        self.algorithmic = cfg.algorithmic_bytes + cfg.B * cfg.k * cfg.V * (4 if cfg.dtype == "f32" else 2)
        self.extra = {"hint": "the gradient of the step before, replaced in place"}

    def step(self, i):
        T, D, x, u = self.sets[i % self.nsets]
        self.res = self.b.sd_verify_feedback_hint(T, D, x, u, self.inp.tau, self.hint, grad_out=self.hint,
                                                  workspace=self.ws)

    def e2e_prepare(self):
        torch, cfg = self.torch, self.cfg
        self.dbuf = [torch.empty_like(t) for t in self.sets[0]]
        self.h_hint = torch.zeros((cfg.B, cfg.k, cfg.V), dtype=self.host[0].dtype).pin_memory()
        self.h_small = [torch.empty(cfg.B, dtype=torch.int32).pin_memory(),
                        torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory(),
                        torch.empty((cfg.B, cfg.k), dtype=torch.float32).pin_memory(),
                        torch.empty((cfg.B, cfg.k), dtype=torch.float32).pin_memory()]
        nbytes = lambda ts: sum(t.numel() * t.element_size() for t in ts)
        self.h2d = self.in_bytes + nbytes([self.h_hint])
        self.d2h = nbytes(self.h_small) + nbytes([self.h_hint])
        self.e2e_entry = "sd_verify_feedback_hint between pinned-memory copies"

    def e2e_step(self):
        for a, b in zip(self.dbuf, self.host):
            a.copy_(b, non_blocking=True)
        self.hint.copy_(self.h_hint, non_blocking=True)
        r = self.b.sd_verify_feedback_hint(*self.dbuf, self.inp.tau, self.hint, grad_out=self.hint, workspace=self.ws)
        for h, d in zip(self.h_small, (r.accept_len, r.tokens, r.loss, r.hint_err)):
            h.copy_(d, non_blocking=True)
        self.h_hint.copy_(self.hint, non_blocking=True)
        self.torch.cuda.synchronize()

    def finish(self, args):
        base, parity, verified = super().finish(args)
        # the hint error of one more step against the oracle on a few sequences (hint = the gradient in place)
        from oracle import sd_oracle
        torch, cfg = self.torch, self.cfg
        seqs = sorted({0, cfg.B // 2, cfg.B - 1})
        T, D, x, u = self.sets[0]
        before = self.hint[seqs].cpu()
        res = self.b.sd_verify_feedback_hint(T, D, x, u, self.inp.tau, self.hint, grad_out=self.hint, workspace=self.ws)
        torch.cuda.synchronize()
        hb = before.view(torch.uint16).numpy() if cfg.dtype == "bf16" else before.numpy()
        want = sd_oracle.hint_error(self.inp.target_logits[seqs], self.inp.draft_logits[seqs], hb, self.inp.tau)
        got = res.hint_err[seqs].cpu().numpy().astype(np.float64)
        ok = bool((np.abs(got - want) <= 1e-3 * want + 1e-12).all())
        parity["hint_error_within_tolerance"] = ok
        return base, parity, bool(verified and ok)


class VocabParallelPath(SamplePath):
    """One rank of the vocabulary-parallel step on this GPU: the workload's logits cut into --shards column
    shards, this rank's three local calls timed on its own shard with the other ranks' records and masses
    already in place (the gathers of a real deployment are not part of the timed region: one GPU here)."""
    name, kernel, traffic_path = "vp", "sd_vp_stats_kernel + sd_vp_rows_kernel + sd_vp_grad_kernel + sd_vp_mass_kernel + sd_vp_draw_kernel", "vp"

    def __init__(self, args, cfg, dev, rank, binding):
        import torch
        from paper_2603_12617_b200 import shard
        self.b, self.cfg, self.torch = binding, cfg, torch
        self.inp = inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
        G = self.G = max(1, args.shards)
        es = cfg.elem_bytes
        self.cuts = cuts = shard.vocab_cuts(cfg.V, G, es)
        code = binding.SD_DTYPE_F32 if cfg.dtype == "f32" else binding.SD_DTYPE_BF16
        T, D = as_torch(inp.target_logits), as_torch(inp.draft_logits)
        x, u = torch.from_numpy(inp.draft_tokens).to(dev), torch.from_numpy(inp.uniforms).to(dev)
        self.x, self.u = x, u
        recs, fins, shards, wss = [], [], [], []
        for r, (a, c) in enumerate(cuts):          # every rank's phases once: what the gathers would deliver
            Ts, Ds = T[:, :, a:c].contiguous().to(dev), D[:, :, a:c].contiguous().to(dev)
            ws = torch.empty(max(256, binding.sd_vp_workspace_bytes(cfg.B, cfg.k, c - a, code)), dtype=torch.uint8, device=dev)
            recs.append(binding.sd_vp_partial(Ts, Ds, x, inp.tau, a, cfg.V, ws))
            shards.append((Ts, Ds)); wss.append(ws)
        self.all_records = torch.stack(recs, 0).contiguous()
        for r, (a, c) in enumerate(cuts):
            fins.append(binding.sd_vp_finish(*shards[r], x, u, inp.tau, a, cfg.V, self.all_records, G, r, wss[r]))
        self.all_masses = torch.stack([f.local_mass for f in fins], 0).contiguous()
        toks = [binding.sd_vp_draw(*shards[r], x, u, inp.tau, cuts[r][0], cfg.V, fins[r].accept_len, self.all_masses,
                                   G, r, fins[r].status, wss[r]) for r in range(G)]
        torch.cuda.synchronize()
        self.check_accept = fins[0].accept_len.cpu().numpy()
        self.check_tokens = torch.stack(toks, 0).max(0).values.cpu().numpy()
        self.check_loss = fins[0].loss.cpu().numpy()
        # the timed rank: rank 0's shard, rotating copies if it is not larger than L2 by itself
        self.host = [shards[0][0].cpu().pin_memory(), shards[0][1].cpu().pin_memory()]
        self.sets, self.in_bytes, self.nsets = rotating_sets(self.host, dev)
        self.ws = wss[0]
        del shards, wss
        Vs = cuts[0][1] - cuts[0][0]
        self.Vs = Vs
        self.algorithmic = (2 * (2 * cfg.k + 1) + cfg.k) * Vs * cfg.B * es
        self.positions = cfg.B * cfg.k
        self.dtype = "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)"
        self.extra = {"shards": G, "timed": f"the three local calls of rank 0 (columns 0..{Vs - 1}); the two gathers and the "
                                           "token maximum of a real deployment are not in the timed region",
                      "kernels_per_step": 5}
        self.e2e_entry = "sd_vp_partial + sd_vp_finish + sd_vp_draw of one rank between pinned-memory copies of its shard"

    def step(self, i):
        Ts, Ds = self.sets[i % self.nsets]
        b, c = self.b, self.cfg
        b.sd_vp_partial(Ts, Ds, self.x, self.inp.tau, 0, c.V, self.ws)
        self.fin = b.sd_vp_finish(Ts, Ds, self.x, self.u, self.inp.tau, 0, c.V, self.all_records, self.G, 0, self.ws)
        self.tok = b.sd_vp_draw(Ts, Ds, self.x, self.u, self.inp.tau, 0, c.V, self.fin.accept_len, self.all_masses, self.G, 0,
                                self.fin.status, self.ws)

    def e2e_prepare(self):
        torch = self.torch
        self.dbuf = [torch.empty_like(t) for t in self.sets[0]]
        self.h_g = torch.empty(self.sets[0][1].shape, dtype=self.host[0].dtype).pin_memory()
        self.h_tok = torch.empty((self.cfg.B, self.cfg.k + 1), dtype=torch.int32).pin_memory()
        self.h2d = self.in_bytes
        self.d2h = self.h_g.numel() * self.h_g.element_size() + self.h_tok.numel() * 4

    def e2e_step(self):
        for a, h in zip(self.dbuf, self.host):
            a.copy_(h, non_blocking=True)
        keep, self.sets, self.nsets = (self.sets, self.nsets), [self.dbuf], 1
        self.step(0)
        self.sets, self.nsets = keep
        self.h_g.copy_(self.fin.grad_shard, non_blocking=True)
        self.h_tok.copy_(self.tok, non_blocking=True)
        self.torch.cuda.synchronize()

    def finish(self, args):
        cfg = self.cfg
        if args.no_cpu_baseline:
            seqs = np.asarray(sorted({0, cfg.B // 2, cfg.B - 1}))
            base, (_, ref) = None, run_oracle(self.inp, seqs, len(seqs), want_grad=False)
        else:
            base, seqs, ref = cpu_baseline(cfg, self.inp)
        parity = parity_counts(cfg, ref, seqs, self.check_accept, self.check_tokens, self.check_loss)
        verified = parity["mismatches_outside_the_bands"] == 0 and parity.get("loss_within_tolerance", True)
        return base, parity, bool(verified)


class GreedyPath:
    name, kernel, traffic_path = "greedy", "sd_greedy_kernel", "greedy"

    def __init__(self, args, cfg, dev, rank, binding):
        import torch
        self.b, self.cfg, self.torch = binding, cfg, torch
        self.inp = inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
        # greedy drafting proposes the draft's argmax; the inputs carry sampled tokens, which serves as well:
        # the work does not depend on the tokens
        self.host = [as_torch(inp.target_logits).pin_memory(), torch.from_numpy(inp.draft_tokens).pin_memory()]
        self.sets, self.in_bytes, self.nsets = rotating_sets(self.host, dev)
        self.out = binding.sd_verify_greedy(*self.sets[0])
        self.algorithmic = (cfg.k + 1) * cfg.V * cfg.B * cfg.elem_bytes
        self.positions = cfg.B * cfg.k
        self.dtype = "f32 comparisons" if cfg.dtype == "f32" else "bf16 comparisons"
        self.extra = {}
        self.e2e_entry = "sd_verify_greedy between pinned-memory copies"

    def step(self, i):
        self.b.sd_verify_greedy(*self.sets[i % self.nsets], out=self.out)

    def e2e_prepare(self):
        torch, cfg = self.torch, self.cfg
        self.dbuf = [torch.empty_like(t) for t in self.sets[0]]
        self.h_n = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        self.h_tok = torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory()
        self.h2d = self.in_bytes
        self.d2h = self.h_n.numel() * 4 + self.h_tok.numel() * 4

    def e2e_step(self):
        for a, b in zip(self.dbuf, self.host):
            a.copy_(b, non_blocking=True)
        self.b.sd_verify_greedy(*self.dbuf, out=self.out)
        self.h_n.copy_(self.out.accept_len, non_blocking=True)
        self.h_tok.copy_(self.out.tokens, non_blocking=True)
        self.torch.cuda.synchronize()

    def finish(self, args):
        from oracle import sd_oracle
        cfg = self.cfg
        t0 = time.perf_counter()
        ref = sd_oracle.verify_greedy(self.inp.target_logits, self.inp.draft_tokens)
        t_cpu = time.perf_counter() - t0
        verified = bool((self.h_n.numpy() == ref.accept_len).all() and (self.h_tok.numpy() == ref.tokens).all()
                        and (self.out.argmax.cpu().numpy() == ref.argmax).all())
        base = {"value": cfg.B * cfg.k / t_cpu, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": f"all {cfg.B} sequences of {cfg.name}, one call, {t_cpu:.2f} s"}
        parity = {"sequences_compared": cfg.B, "mismatches_outside_the_bands": 0 if verified else None,
                  "mean_accept_len": float(self.h_n.float().mean())}
        return base, parity, verified


class ErrorsPath:
    name, kernel, traffic_path = "errors", "sd_stream_kernel<pass 1 only> + sd_errpos_kernel", "errors"

    def __init__(self, args, cfg, dev, rank, binding):
        import torch
        self.b, self.cfg, self.torch = binding, cfg, torch
        self.inp = inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
        self.host = [as_torch(inp.target_logits).pin_memory(), as_torch(inp.draft_logits).pin_memory(),
                     torch.from_numpy(inp.draft_tokens).pin_memory(), torch.from_numpy(inp.uniforms).pin_memory()]
        self.sets, self.in_bytes, self.nsets = rotating_sets(self.host, dev)
        self.out = binding.sd_verify_error_feedback(*self.sets[0], inp.tau)
        self.algorithmic = ((2 * cfg.k + 1) + 1) * cfg.V * cfg.B * cfg.elem_bytes
        self.positions = cfg.B * cfg.k
        self.dtype = "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)"
        self.extra = {}
        self.e2e_entry = "sd_verify_error_feedback between pinned-memory copies"

    def step(self, i):
        self.b.sd_verify_error_feedback(*self.sets[i % self.nsets], self.inp.tau, out=self.out)

    def e2e_prepare(self):
        torch, cfg = self.torch, self.cfg
        self.dbuf = [torch.empty_like(t) for t in self.sets[0]]
        self.h_n = torch.empty(cfg.B, dtype=torch.int32).pin_memory()
        self.h_tok = torch.empty((cfg.B, cfg.k + 1), dtype=torch.int32).pin_memory()
        self.h_loss = torch.empty((cfg.B, cfg.k), dtype=torch.float32).pin_memory()
        self.h_g = torch.empty((cfg.B, cfg.V), dtype=self.host[0].dtype).pin_memory()
        self.h2d = self.in_bytes
        self.d2h = self.h_n.numel() * 4 + self.h_tok.numel() * 4 + self.h_loss.numel() * 4 + self.h_g.numel() * self.h_g.element_size()

    def e2e_step(self):
        for a, b in zip(self.dbuf, self.host):
            a.copy_(b, non_blocking=True)
        self.b.sd_verify_error_feedback(*self.dbuf, self.inp.tau, out=self.out)
        self.h_n.copy_(self.out.accept_len, non_blocking=True)
        self.h_tok.copy_(self.out.tokens, non_blocking=True)
        self.h_loss.copy_(self.out.loss, non_blocking=True)
        self.h_g.copy_(self.out.error_grad, non_blocking=True)
        self.torch.cuda.synchronize()

    def finish(self, args):
        from oracle import sd_oracle
        cfg, inp = self.cfg, self.inp
        cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
        nseq = min(cfg.B, cores)
        sl = np.arange(nseq)
        t0 = time.perf_counter()
        ref = sd_oracle.error_position_feedback(inp.target_logits[sl], inp.draft_logits[sl], inp.draft_tokens[sl],
                                                inp.uniforms[sl], inp.tau, nthreads=cores)
        t_cpu = time.perf_counter() - t0
        parity = parity_counts(cfg, ref.full, sl, self.h_n.numpy(), self.h_tok.numpy(), self.h_loss.numpy())
        safe = (ref.full.accept_band.sum(1) == 0) & (ref.full.cdf_margin > 1e-6)
        g = self.h_g[:nseq].float().numpy().astype(np.float64)
        tol = TOL[cfg.dtype]
        grads_ok = all(np.abs(g[b] - ref.error_grad[b]).max() <= tol * np.abs(ref.error_grad[b]).max() + 1e-6
                       for b in range(nseq) if safe[b])
        verified = bool(parity["mismatches_outside_the_bands"] == 0 and parity["loss_within_tolerance"] and grads_ok)
        base = {"value": nseq * cfg.k / t_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"{nseq} of {cfg.B} sequences of {cfg.name}, one call, {t_cpu:.2f} s"}
        return base, parity, verified


class EnsemblePath:
    name, kernel, traffic_path = "ensemble", "sd_stream_kernel<ensemble> + sd_hedge_kernel", "ensemble"
    EPS = 10.0

    def __init__(self, args, cfg, dev, rank, binding):
        import torch
        self.b, self.cfg, self.torch = binding, cfg, torch
        self.N = N = args.learners
        self.inp = inp = synth.make_inputs(cfg, seed=synth.BASE_SEED + 1000 * rank)
        self.drafts = synth.ensemble_drafts(inp, N, seed=synth.BASE_SEED + 1000 * rank)
        self.host = [as_torch(inp.target_logits).pin_memory()] + [as_torch(d).pin_memory() for d in self.drafts]
        self.sets, self.in_bytes, self.nsets = rotating_sets(self.host, dev)
        self.out = binding.sd_ensemble_feedback(self.sets[0][0], self.sets[0][1:], inp.tau, self.EPS)
        self.cum = torch.zeros(N, dtype=torch.float64, device=dev)
        self.algorithmic = ((cfg.k + N * cfg.k) + N * cfg.k) * cfg.V * cfg.B * cfg.elem_bytes
        self.positions = cfg.B * cfg.k
        self.dtype = "f32" if cfg.dtype == "f32" else "f32 (bf16 storage)"
        self.extra = {"learners": N, "epsilon": self.EPS}
        self.traffic_extra = str(N)
        self.e2e_entry = "sd_ensemble_feedback between pinned-memory copies"

    def step(self, i):
        s = self.sets[i % self.nsets]
        self.b.sd_ensemble_feedback(s[0], s[1:], self.inp.tau, self.EPS, cum_loss=self.cum, out=self.out)

    def e2e_prepare(self):
        torch, cfg, N = self.torch, self.cfg, self.N
        self.dbuf = [torch.empty_like(t) for t in self.sets[0]]
        self.h_loss = torch.empty((N, cfg.B, cfg.k), dtype=torch.float32).pin_memory()
        self.h_w = torch.empty(N, dtype=torch.float32).pin_memory()
        self.h_grad = [torch.empty_like(d).pin_memory() for d in self.host[1:]]
        self.h2d = self.in_bytes
        self.d2h = self.h_loss.numel() * 4 + self.h_w.numel() * 4 + sum(g.numel() * g.element_size() for g in self.h_grad)

    def e2e_step(self):
        for a, b in zip(self.dbuf, self.host):
            a.copy_(b, non_blocking=True)
        self.b.sd_ensemble_feedback(self.dbuf[0], self.dbuf[1:], self.inp.tau, self.EPS, cum_loss=self.cum, out=self.out)
        self.h_loss.copy_(self.out.loss, non_blocking=True)
        self.h_w.copy_(self.out.weights, non_blocking=True)
        for a, b in zip(self.h_grad, self.out.grad):
            a.copy_(b, non_blocking=True)
        self.torch.cuda.synchronize()

    def finish(self, args):
        from oracle import sd_oracle
        cfg, inp, N = self.cfg, self.inp, self.N
        cores = min(sd_oracle.max_threads(), os.cpu_count() or 1)
        nseq = min(cfg.B, max(1, cores // cfg.k))
        sl = np.arange(nseq)
        t0 = time.perf_counter()
        ref = sd_oracle.ensemble_feedback(inp.target_logits[sl], [d[sl] for d in self.drafts], inp.tau, self.EPS,
                                          want_grad=False, nthreads=cores)
        t_cpu = time.perf_counter() - t0
        loss = self.h_loss.numpy()[:, :nseq].astype(np.float64)
        ok = bool((np.abs(loss - ref.loss) <= TOL[cfg.dtype] * np.maximum(np.abs(ref.loss), 1e-6)).all()
                  and abs(float(self.h_w.sum()) - 1.0) < 1e-5)
        base = {"value": nseq * cfg.k / t_cpu, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"{nseq} of {cfg.B} sequences of {cfg.name}, {N} learners, no gradients, one call, {t_cpu:.2f} s"}
        parity = {"sequences_compared": int(nseq), "loss_within_tolerance": ok}
        return base, parity, ok


class LmHeadPath:
    """The step after the path: dW = g^T X for the R = B*k positions of the workload."""
    name, kernel, traffic_path = "lmhead", "sd_lmhead_kernel", "lmhead"

    def __init__(self, args, cfg, dev, rank, binding):
        import torch
        self.b, self.cfg, self.torch = binding, cfg, torch
        self.R, self.V, self.d = cfg.B * cfg.k, cfg.V, args.features
        gb, Xb = synth.lmhead_operands(self.R, self.V, self.d, seed=synth.BASE_SEED + 1000 * rank)
        self.gb, self.Xb = gb, Xb
        self.host = [as_torch(gb).pin_memory(), as_torch(Xb).pin_memory()]
        self.sets, self.in_bytes, self.nsets = rotating_sets(self.host, dev)
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.out = torch.empty((self.V, self.d), dtype=torch.float32, device=dev)
        self.algorithmic = 2 * self.R * self.V * self.d         # flops
        self.positions = self.R
        self.dtype = "bf16 operands, f32 accumulation"
        self.extra = {"features": self.d, "positions": self.R}
        self.e2e_entry = "sd_lmhead_grad between pinned-memory copies"
        self.bound = "tensor"

    def step(self, i):
        g, X = self.sets[i % self.nsets]
        self.b.sd_lmhead_grad(g, X, out=self.out, status=self.status)

    def e2e_prepare(self):
        torch = self.torch
        self.dbuf = [torch.empty_like(t) for t in self.sets[0]]
        self.h_out = torch.empty((self.V, self.d), dtype=torch.float32).pin_memory()
        self.h2d = self.in_bytes
        self.d2h = self.h_out.numel() * 4

    def e2e_step(self):
        for a, b in zip(self.dbuf, self.host):
            a.copy_(b, non_blocking=True)
        self.b.sd_lmhead_grad(*self.dbuf, out=self.out, status=self.status)
        self.h_out.copy_(self.out, non_blocking=True)
        self.torch.cuda.synchronize()

    def finish(self, args):
        from oracle import sd_oracle
        rng = np.random.default_rng(11)
        n = 4000
        vs, js = rng.integers(0, self.V, n), rng.integers(0, self.d, n)
        t0 = time.perf_counter()
        ref = sd_oracle.lmhead_grad(self.gb, self.Xb, vs, js)
        t_cpu = time.perf_counter() - t0
        got = self.h_out.numpy()[vs, js].astype(np.float64)
        g = np.abs(synth.bf16_bits_to_f32(self.gb).astype(np.float64))
        X = np.abs(synth.bf16_bits_to_f32(self.Xb).astype(np.float64))
        bound = 2e-5 * np.einsum("re,re->e", g[:, vs], X[:, js]) + 1e-30
        ok = bool((np.abs(got - ref) <= bound).all() and int(self.status.item()) == 0)
        full_s = t_cpu * (self.V * self.d / n)
        base = {"value": self.R / full_s, "unit": UNIT, "cores": 1, "kind": "oracle",
                "sample": f"{n} of {self.V * self.d} entries of dW, {t_cpu:.2f} s, scaled to all of dW"}
        return base, {"entries_compared": n, "within_tolerance": ok}, ok


PATHS = {"sample": SamplePath, "hint": HintPath, "vp": VocabParallelPath, "greedy": GreedyPath, "errors": ErrorsPath, "ensemble": EnsemblePath, "lmhead": LmHeadPath}


def run_ours(args, cfg):
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

    # every rank works on a full batch of its own (different seed per rank): weak scaling
    path = PATHS[args.path](args, cfg, dev, rank, binding)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    warmup = max(3, args.warmup)
    for i in range(warmup):
        path.step(i)
    info = binding.sd_launch_info()
    barrier()
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # The launching thread gets a head start: the stream first spins on the device for about as long
    # as it takes the host to enqueue every step, so that the steps run back to back and neither the
    # step time nor the per-launch times below contain the host's launch latency (on the small
    # workloads enqueueing a step takes longer than running it).  The spin ends before t_begin.
    head_ms = min(60.0, max(2.0, 0.08 * args.steps))
    sm_khz = torch.cuda.get_device_properties(local).clock_rate if hasattr(
        torch.cuda.get_device_properties(local), "clock_rate") else 1_900_000
    with ClockSampler(local) as clocks:
        torch.cuda._sleep(int(head_ms * sm_khz))
        t_begin.record()
        for i in range(args.steps):
            starts[i].record()
            path.step(i)
            ends[i].record()
        t_end.record()
        clocks.sample_now()                   # the queue is still full of work: the GPU is under load here
        barrier()
    dev_arg = str(dev) if world > 1 else "cpu"
    total_ms = shard.max_over_ranks(t_begin.elapsed_time(t_end), device=dev_arg)
    kernel_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    mean_kernel_ms = float(np.mean(kernel_ms))
    if args.times_out and rank == 0:
        with open(args.times_out, "w") as fh:
            json.dump(kernel_ms, fh)
    positions = path.positions * world
    value = positions * args.steps / (total_ms * 1e-3)

    # end to end: pinned host buffers in, host buffers out, every copy inside the timed region
    e2e_steps = max(1, min(args.steps, 3 if args.path == "lmhead" else 10))
    path.e2e_prepare()
    for _ in range(2):
        path.e2e_step()
    barrier()
    t0 = time.perf_counter()
    for _ in range(e2e_steps):
        path.e2e_step()
    barrier()
    e2e_s = shard.max_over_ranks(time.perf_counter() - t0, device=dev_arg)
    e2e = {"value": positions * e2e_steps / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(path.h2d),
           "d2h_bytes_per_step": int(path.d2h), "steps": e2e_steps, "ms_per_step": e2e_s / e2e_steps * 1e3,
           "entry_point": path.e2e_entry}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    if getattr(path, "bound", "hbm") == "tensor":
        achieved = path.algorithmic / (mean_kernel_ms * 1e-3) / 1e12
        long_run = args.steps * mean_kernel_ms > 2000.0
        peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
        roofline = {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                    "traffic": None, "peak_source": peaks["source"] + (", sustained figure (timed region over 2 s)" if long_run else ", burst figure"),
                    "flops_per_launch": path.algorithmic, "kernel_ms_mean": mean_kernel_ms,
                    "kernel_ms_min": float(np.min(kernel_ms)), "kernel": path.kernel}
    else:
        achieved = path.algorithmic / (mean_kernel_ms * 1e-3) / 1e9
        traffic, traffic_source = (None, "not the full-size workload") if args.batch else \
            captured_traffic(path.traffic_path, cfg.name, getattr(path, "traffic_extra", "-"))
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": achieved / peaks["hbm_gbs"], "traffic": traffic, "traffic_source": traffic_source,
                    "peak_source": peaks["source"], "algorithmic_bytes_per_launch": path.algorithmic,
                    "kernel_ms_mean": mean_kernel_ms, "kernel_ms_min": float(np.min(kernel_ms)),
                    "kernel": path.kernel if info["path"] != 0 else "sd_generic_kernel",
                    "frac_of_nominal_8000_GBps": achieved / 8000.0}
    base, parity, verified = path.finish(args)
    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": path.dtype, "data": "synthetic",
            "config": workload_config(cfg, path=args.path,
                                      l2="inputs larger than L2" if path.nsets == 1 else f"{path.nsets} rotating input sets larger than L2 together",
                                      parallelism=f"replicas x{world}, sequences independent, no collective",
                                      launch=info, **path.extra),
            "roofline": roofline, "cpu_baseline": base, "e2e": e2e,
            "gpu_launches": args.steps * int(path.extra.get("kernels_per_step", info["kernels"])),
            "clocks": clocks.summary(), "parity": parity, "outputs_verified_against_oracle": verified}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------
def free_port() -> int:
    with socket.socket(socket.AF_INET, socket.SOCK_STREAM) as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launcher_command(argv, gpus: int, port: int):
    """The command that starts one rank per GPU on this node for `python bench.py <argv>`."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default="cfg5", choices=sorted(synth.CONFIGS))
    ap.add_argument("--batch", type=int, default=0, help="override B (profiling on a smaller case)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--path", choices=sorted(PATHS), default="sample",
                    help="sample: the verify-and-feedback step (the headline); the others: see the module text")
    ap.add_argument("--learners", type=int, default=3, help="draft models of --path ensemble")
    ap.add_argument("--shards", type=int, default=4, help="column shards of --path vp (one rank of them is timed)")
    ap.add_argument("--features", type=int, default=4096, help="width d of the output layer of --path lmhead")
    ap.add_argument("--times-out", default="", help="write the per-step device times (ms) here")
    args = ap.parse_args(argv)
    cfg = synth.CONFIGS[args.config]
    if args.batch:
        cfg = cfg.with_batch(args.batch)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # not started by torch.distributed.run: start one rank per GPU ourselves (the ranks print; rank 0 the line)
        env = dict(os.environ)
        env.setdefault("NCCL_DEBUG", "INFO")      # the communicator's rank count shows in the log (stderr)
        raise SystemExit(subprocess.call(launcher_command(argv, args.gpus, free_port()), env=env))
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the DVM hot path on B200.

One "step" = one pass over a whole dynamic-shape sweep: every instance is
re-encoded on the host (dvm_encode) and launched (dvm_launch /
dvm_launch_stacked); nothing is cached between instances.  The default
workload is the fused residual-add + RMSNorm sweep (200 instances, bf16
[B*S, 4096], B in 1..32, S in 1..8192).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c1|c2|c3|c4|c5|addmm|ifelse|views] [--impl dvm|reference]

Prints one JSON line (rank 0).  The default run (c2) also measures every other workload briefly and reports
them under `configs` (throughput, roofline fraction, launches; --no-configs leaves that out).  `value` is algorithmic GB/s of the whole job
with inputs resident in HBM; `e2e` is the same metric through dvm_run_host
with pinned HOST buffers (copies inside the timed region); `roofline` is the
interpreter kernel's algorithmic bytes over its CUDA-event time against the
measured HBM copy peak; `cpu_baseline` is the CPU oracle timed on a bounded
sample on this machine's host cores.
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

import numpy as np
import torch

import dvm_workloads as wl

FALLBACK_HBM_GBS = 6650.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return json.load(f), "measured"
    except Exception:
        return {"hbm_gbs": FALLBACK_HBM_GBS, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}, "fallback"


# ----------------------------------------------------------------------------- clocks
class ClockSampler:
    """Samples nvidia-smi clocks / throttle reasons of one GPU while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w_max": max(power) if power else None, "samples": len(sm), "reasons": sorted(reasons)}


# ----------------------------------------------------------------------------- workloads
class C1Workload:
    """Single fused elementwise program out = exp(a*b + c) - a, fp32 [7,1531], seed 0 (config 1): launch-latency bound."""
    name = "c1"

    def __init__(self, dvm, n_instances=1, device="cuda"):
        self.dvm = dvm
        self.prog = wl.program_c1()
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.ins = wl.inputs_c1(device)
        self.out = torch.empty((7, 1531), dtype=torch.float32, device=device)
        self.n = max(1, n_instances)
        self.bytes_per_instance = [16 * 7 * 1531] * self.n
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = ("c1: out = exp(a*b + c) - a, fp32 [7,1531] U(-1,1) seed 0, encoded and launched once per step "
                            "(171 KB: launch-latency bound; the figure of merit is microseconds per launch)")
        self.l2_policy = "171 KB working set: L2-resident by nature; no roofline claim"

    def run_step(self, stream, events=None, enc_ns=None):
        import ctypes as C
        lib_launch = self.dvm.binding.lib.dvm_launch
        for _ in range(self.n):
            t0 = time.perf_counter_ns()
            size = self.enc.encode(((7, 1531),) * 3)
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            arr = (C.c_void_p * 4)(*[t.data_ptr() for t in self.ins], self.out.data_ptr())
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(self.enc.buf, size, arr, 4, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return self.n

    def setup_e2e(self):
        self.h_in = [t.cpu().pin_memory() for t in self.ins]
        self.h_out = torch.empty((7, 1531), dtype=torch.float32).pin_memory()
        self.staging = torch.empty(4 * 7 * 1531 * 4 + 4 * 256, dtype=torch.uint8, device="cuda")

    def run_step_e2e(self, stream):
        self.enc.encode(((7, 1531),) * 3)
        code = self.dvm.Code(self.enc.buf, self.enc.size.value, None)
        h2d = d2h = 0
        for _ in range(self.n):
            self.dvm.run_host(code, self.h_in + [self.h_out], self.staging, stream)
            h2d += 3 * 7 * 1531 * 4
            d2h += 7 * 1531 * 4
        return h2d, d2h

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        ins = [wl.to_f64(t) for t in self.ins]
        t0 = time.perf_counter(); k = 0
        while time.perf_counter() - t0 < budget_s:
            orc.evaluate(self.prog.nodes, ins); k += 1
        dt = time.perf_counter() - t0
        return k * 16 * 7 * 1531 / dt / 1e9, dt, f"{k} evaluations of the [7,1531] instance, numpy float64"


class C2Workload:
    """Fused residual-add + RMSNorm, bf16 [B*S, 4096], 200 dynamic instances (config 2)."""
    name = "c2"
    hidden = 4096

    def __init__(self, dvm, n_instances=200, device="cuda", max_rows=0):
        self.dvm = dvm
        self.prog = wl.program_add_rmsnorm(self.hidden)
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.shapes = wl.shapes_c2(n_instances)
        self.rows = [b * s for b, s in self.shapes]
        if max_rows:
            self.rows = [min(r, max_rows) for r in self.rows]
        self.pool_rows = max(self.rows)
        H = self.hidden
        seed = wl.data_seed("c2", 0)
        # inputs resident in HBM: one pool per tensor, instances take rotating row windows
        self.x = wl.randn((self.pool_rows, H), torch.bfloat16, seed, device)
        self.res = wl.randn((self.pool_rows, H), torch.bfloat16, seed + 7919, device)
        self.w = wl.randn((H,), torch.bfloat16, seed + 104729, device, mean=1.0, std=0.02)
        self.y = torch.empty((self.pool_rows, H), dtype=torch.bfloat16, device=device)
        self.h = torch.empty((self.pool_rows, H), dtype=torch.bfloat16, device=device)
        self.offsets = []
        off = 0
        for t in self.rows:
            if off + t > self.pool_rows:
                off = 0
            self.offsets.append(off)
            off += t
        self.bytes_per_instance = [t * H * 8 + H * 2 for t in self.rows]
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = ("c2: fused residual-add + RMSNorm (eps 1e-6), bf16 [B*S,4096], fp32 internal, "
                            f"{n_instances} dynamic instances (B 1..32, S 1..8192), each re-encoded per launch")
        self.l2_policy = ("inputs >> L2: mean 2.2 GB per instance, rotating row windows over 2 GiB pools "
                          "per tensor")

    def tensors(self, i):
        o, t = self.offsets[i], self.rows[i]
        return [self.x[o:o + t], self.res[o:o + t], self.w, self.y[o:o + t], self.h[o:o + t]]

    def run_step(self, stream, events=None, enc_ns=None):
        """One pass over the sweep.  events: optional list to receive (start, end) per launch."""
        dvm, enc = self.dvm, self.enc
        H = self.hidden
        lib_launch = dvm.binding.lib.dvm_launch
        import ctypes as C
        for i, t in enumerate(self.rows):
            t0 = time.perf_counter_ns()
            size = enc.encode(((t, H), (t, H), (H,)))
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            ts = self.tensors(i)
            arr = (C.c_void_p * 5)(*[x.data_ptr() for x in ts])
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(enc.buf, size, arr, 5, stream.cuda_stream)
            if st != 0:
                raise dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.rows)

    # ---- end to end with host buffers -------------------------------------------------
    def setup_e2e(self):
        H = self.hidden
        n = self.pool_rows
        self.hx = torch.empty((n, H), dtype=torch.bfloat16).pin_memory()
        self.hres = torch.empty((n, H), dtype=torch.bfloat16).pin_memory()
        self.hw = self.w.cpu().pin_memory()
        self.hy = torch.empty((n, H), dtype=torch.bfloat16).pin_memory()
        self.hh = torch.empty((n, H), dtype=torch.bfloat16).pin_memory()
        self.hx.copy_(self.x); self.hres.copy_(self.res)
        self.staging = torch.empty(4 * n * H * 2 + H * 2 + 5 * 256, dtype=torch.uint8, device="cuda")

    def run_step_e2e(self, stream):
        H = self.hidden
        h2d = d2h = 0
        for i, t in enumerate(self.rows):
            o = self.offsets[i]
            self.enc.encode(((t, H), (t, H), (H,)))
            code = self.dvm.Code(self.enc.buf, self.enc.size.value, None)
            host = [self.hx[o:o + t], self.hres[o:o + t], self.hw, self.hy[o:o + t], self.hh[o:o + t]]
            self.dvm.run_host(code, host, self.staging, stream)
            h2d += 2 * t * H * 2 + H * 2
            d2h += 2 * t * H * 2
        return h2d, d2h

    # ---- CPU oracle on a bounded sample ------------------------------------------------
    def oracle_sample(self, budget_s=12.0):
        """The oracle on every host core: each worker process evaluates its own window of 1024 rows of the pools."""
        from oracle import parallel as opar
        H = self.hidden
        w = wl.to_f64(self.w)
        rows = min(1024, self.pool_rows)
        n_win = max(1, min(os.cpu_count() or 1, self.pool_rows // rows))
        cases = [[wl.to_f64(self.x[k * rows:(k + 1) * rows]), wl.to_f64(self.res[k * rows:(k + 1) * rows]), w] for k in range(n_win)]
        done, dt, n = opar.evaluate_on_all_cores(self.prog.nodes, cases, (), budget_s)
        self.oracle_cores = n
        nbytes = done * (rows * H * 8 + H * 2)
        return nbytes / dt / 1e9, dt, (f"{done} evaluations of windows of {rows} rows x {H} of the c2 pools, numpy float64, "
                                       f"{n} worker processes (one per host core), total work over the slowest worker's time")


class C3Workload:
    """Masked softmax over attention scores bf16 [B,32,S,S] (config 3), 100 dynamic instances."""
    name = "c3"
    heads = 32

    def __init__(self, dvm, n_instances=100, device="cuda"):
        self.dvm = dvm
        self.prog = wl.program_masked_softmax(128)
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.shapes = wl.shapes_c3(n_instances)
        self.elems = [b * self.heads * s * s for b, s in self.shapes]
        self.pool = max(self.elems)
        seed = wl.data_seed("c3", 0)
        self.scores = wl.randn((self.pool,), torch.bfloat16, seed, device)
        self.out = torch.empty((self.pool,), dtype=torch.bfloat16, device=device)
        self.masks = {s: wl.causal_mask(s, device) for s in sorted({s for _, s in self.shapes})}
        self.offsets = []
        off = 0
        for n in self.elems:
            n8 = (n + 127) // 128 * 128
            if off + n8 > self.pool:
                off = 0
            self.offsets.append(off)
            off += n8
        self.bytes_per_instance = [n * 4 + 2 * s * s for n, (_, s) in zip(self.elems, self.shapes)]
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = ("c3: (scores + causal mask) / sqrt(128), row softmax, bf16 [B,32,S,S], fp32 internal, "
                            f"{n_instances} dynamic instances (B 1..8, S 17..2048), each re-encoded per launch")
        self.l2_policy = "inputs >> L2: mean 0.8 GB per instance, rotating windows over a 2 GiB pool"

    def run_step(self, stream, events=None, enc_ns=None):
        import ctypes as C
        lib_launch = self.dvm.binding.lib.dvm_launch
        Hh = self.heads
        for i, (b, s) in enumerate(self.shapes):
            t0 = time.perf_counter_ns()
            size = self.enc.encode(((b, Hh, s, s), (1, 1, s, s)))
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            o, n = self.offsets[i], self.elems[i]
            arr = (C.c_void_p * 3)(self.scores.data_ptr() + 2 * o, self.masks[s].data_ptr(),
                                   self.out.data_ptr() + 2 * o)
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(self.enc.buf, size, arr, 3, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.shapes)

    def setup_e2e(self):
        self.hs = torch.empty((self.pool,), dtype=torch.bfloat16).pin_memory()
        self.ho = torch.empty((self.pool,), dtype=torch.bfloat16).pin_memory()
        self.hs.copy_(self.scores)
        self.hmasks = {s: m.cpu().pin_memory() for s, m in self.masks.items()}
        self.staging = torch.empty(2 * self.pool * 2 + 2048 * 2048 * 2 + 4 * 256, dtype=torch.uint8, device="cuda")

    def run_step_e2e(self, stream):
        h2d = d2h = 0
        Hh = self.heads
        for i, (b, s) in enumerate(self.shapes):
            self.enc.encode(((b, Hh, s, s), (1, 1, s, s)))
            code = self.dvm.Code(self.enc.buf, self.enc.size.value, None)
            o, n = self.offsets[i], self.elems[i]
            host = [self.hs[o:o + n], self.hmasks[s], self.ho[o:o + n]]
            self.dvm.run_host(code, host, self.staging, stream)
            h2d += 2 * n + 2 * s * s
            d2h += 2 * n
        return h2d, d2h

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        S, B, Hh = 512, 1, 8
        n = B * Hh * S * S
        m = wl.to_f64(wl.causal_mask(S))
        t_all, done, off = 0.0, 0, 0
        while t_all < budget_s:
            if off + n > self.pool:
                off = 0
            sc = wl.to_f64(self.scores[off:off + n]).reshape(B, Hh, S, S)
            t0 = time.perf_counter(); orc.evaluate(self.prog.nodes, [sc, m]); t_all += time.perf_counter() - t0
            done += 1; off += n
        return done * (n * 4 + 2 * S * S) / t_all / 1e9, t_all, f"{done} instances of scores [1,{Hh},{S},{S}] from the c3 pool, numpy float64"


class C4Workload:
    """Stacking-based fusion: 64 independent small fp32 programs per launch, 50 launches (config 4)."""
    name = "c4"

    def __init__(self, dvm, n_launches=50, device="cuda"):
        self.dvm = dvm
        # Programs of one stacked launch share the elements-per-thread setting, and the launch's CTAs are sized by
        # its largest program.  32 elements per thread halve the per-tile overhead per element; two tile slots of that
        # size fit an SM once, so the launch runs with ONE slot per CTA, two CTAs per SM (measured on this sweep:
        # 16 elements / two slots 2007 GB/s kernel-only, 32 / two slots 1809, 16 / one slot 1622, 32 / one slot 2268).
        if not dvm.binding.lib.dvm_get_elems_per_thread():
            dvm.set_elems_per_thread(32)
        dvm.set_min_resident_ctas(3)
        dvm.set_stacked_one_slot(True)
        self.launches = wl.shapes_c4(n_launches)
        self.progs = {k: wl.stack_program(k) for k in wl.STACK_KINDS}
        self.ps = {k: dvm.program_from_nodes(p.nodes) for k, p in self.progs.items()}
        # distinct buffers for every program of every launch (~16 GB): nothing is reused between launches
        self.items = []
        seed = wl.data_seed("c4", 0)
        nbytes = 0
        for li, launch in enumerate(self.launches):
            row = []
            for pi, (kind, r, c) in enumerate(launch):
                ins, params = wl.inputs_stack(kind, r, c, seed + li * 64 * 4 + pi * 4, device)
                out = torch.empty((r, c), dtype=torch.float32, device=device)
                per = {"gelu_affine": 8 * r * c + 8 * c, "layernorm": 8 * r * c, "sigmoid_mul": 12 * r * c}[kind]
                nbytes += per
                row.append((kind, r, c, ins, params, out, per))
            self.items.append(row)
        self.total_bytes = nbytes
        self.bytes_per_instance = [sum(it[6] for it in row) for row in self.items]
        self.description = ("c4: stacking-based fusion, 64 independent fp32 programs per launch "
                            "(GELU(x*w+b) / LayerNorm / sigmoid(x)*y, rows 1..512, cols 64..4096), "
                            f"{n_launches} launches, every program re-encoded per launch")
        self.l2_policy = "every launch reads buffers of its own (16 GB in total, ~320 MB per launch > L2)"

    def _launch_args(self, li):
        """Per launch (set up once): the batch encoder over its 64 programs and the tensor pointer tables."""
        import ctypes as C
        row = self.items[li]
        be = self.dvm.binding.BatchEncoder([self.ps[kind] for (kind, *_rest) in row])
        n = len(row)
        keep = [(C.c_void_p * (len(ins) + 1))(*[t.data_ptr() for t in ins], out.data_ptr())
                for (_k, _r, _c, ins, _p, out, _b) in row]
        tptr = (C.POINTER(C.c_void_p) * n)(*[C.cast(a, C.POINTER(C.c_void_p)) for a in keep])
        nt = (C.c_int * n)(*[len(it[3]) + 1 for it in row])
        shapes = [[tuple(t.shape) for t in it[3]] for it in row]
        scalars = [list(it[4]) for it in row]
        return be, tptr, nt, keep, shapes, scalars

    def run_step(self, stream, events=None, enc_ns=None):
        lib = self.dvm.binding.lib
        if not hasattr(self, "_args"):
            self._args = [self._launch_args(li) for li in range(len(self.items))]
        for be, tptr, nt, _keep, shapes, scalars in self._args:
            t0 = time.perf_counter_ns()
            be.encode(shapes, scalars)   # every program of the launch is re-encoded: one dvm_encode_batch call
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append((t1 - t0) / be.n)   # per program
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib.dvm_launch_stacked(be.n, be.codes, be.sizes, tptr, nt, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch_stacked")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.items)

    E2E_LAUNCHES = 10   # end to end runs the first launches only (pinned host copies of all 16 GB would not pay)

    def setup_e2e(self):
        n = min(self.E2E_LAUNCHES, len(self.items))
        self.h_in = [[[t.cpu().pin_memory() for t in it[3]] for it in row] for row in self.items[:n]]
        self.h_out = [[torch.empty(it[5].shape, dtype=torch.float32).pin_memory() for it in row] for row in self.items[:n]]
        self.e2e_work = sum(self.bytes_per_instance[:n])
        self.staging = True

    def run_step_e2e(self, stream):
        """Per launch: pinned host -> device copies of every input, one dvm_launch_stacked, device -> pinned host
        copies of every output, stream sync."""
        lib = self.dvm.binding.lib
        h2d = d2h = 0
        for li, (h_in, h_out) in enumerate(zip(self.h_in, self.h_out)):
            be, tptr, nt, _keep, shapes, scalars = self._args[li]
            row = self.items[li]
            for it, hin in zip(row, h_in):
                for d, h in zip(it[3], hin):
                    d.copy_(h, non_blocking=True)
                    h2d += h.numel() * 4
            be.encode(shapes, scalars)
            st = lib.dvm_launch_stacked(be.n, be.codes, be.sizes, tptr, nt, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch_stacked")
            for it, ho in zip(row, h_out):
                ho.copy_(it[5], non_blocking=True)
                d2h += ho.numel() * 4
            stream.synchronize()
        return h2d, d2h

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        t0 = time.perf_counter()
        nbytes, k = 0, 0
        for row in self.items:
            for (kind, r, c, ins, params, out, per) in row:
                orc.evaluate(self.progs[kind].nodes, [wl.to_f64(t) for t in ins], params)
                nbytes += per; k += 1
                if time.perf_counter() - t0 > budget_s:
                    break
            if time.perf_counter() - t0 > budget_s:
                break
        dt = time.perf_counter() - t0
        return nbytes / dt / 1e9, dt, f"first {k} programs of the sweep (launch 0 onwards), numpy float64, input widening included"


class C5Workload:
    """LLM MLP gate SiLU(X Wg) * (X Wu), bf16 X [M,4096], W [4096,11008] x2, fp32 accumulate, bf16 out (config 5)."""
    name = "c5"
    K, N = 4096, 11008
    metric, unit, scale, bound, kernel, peak_key = "tflops_dynamic_shape_sweep", "TFLOP/s", 1e12, "tensor", "dvm_mm_kernel", "bf16_tflops_sustained"

    def __init__(self, dvm, n_instances=64, device="cuda", max_rows=0):
        self.dvm = dvm
        self.prog = wl.program_mlp_gate()
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.Ms = wl.shapes_c5(n_instances)
        if max_rows:
            self.Ms = [min(m, max_rows) for m in self.Ms]
        K, N = self.K, self.N
        self.wg, self.wu = wl.mlp_weights(K, N, device)      # generated once, reused by every instance
        self.pool_rows = max(self.Ms)
        self.x = wl.randn((self.pool_rows, K), torch.bfloat16, wl.data_seed("c5", 0), device)
        self.out = torch.empty((self.pool_rows, N), dtype=torch.bfloat16, device=device)
        self.work_per_instance = [4 * m * K * N for m in self.Ms]          # two matmuls, 2 flops per multiply-add
        self.bytes_per_instance = [2 * K * N * 2 + m * K * 2 + m * N * 2 for m in self.Ms]
        self.total_work = sum(self.work_per_instance)
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = ("c5: MLP gate SiLU(X Wg) * (X Wu), bf16 X [M,4096] x W [4096,11008] x2 (row-major), fp32 "
                            f"accumulate, bf16 out, {n_instances} dynamic instances (M 1..4096), each re-encoded per launch")
        self.l2_policy = "every instance streams both weight matrices (180 MB > L2) plus its own X / out windows"

    def run_step(self, stream, events=None, enc_ns=None):
        import ctypes as C
        lib_launch = self.dvm.binding.lib.dvm_launch
        K, N = self.K, self.N
        for m in self.Ms:
            t0 = time.perf_counter_ns()
            size = self.enc.encode(((m, K), (K, N), (K, N)))
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            arr = (C.c_void_p * 4)(self.x.data_ptr(), self.wg.data_ptr(), self.wu.data_ptr(), self.out.data_ptr())
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(self.enc.buf, size, arr, 4, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.Ms)

    def setup_e2e(self):
        K, N = self.K, self.N
        self.hx = self.x.cpu().pin_memory()
        self.hwg = self.wg.cpu().pin_memory()
        self.hwu = self.wu.cpu().pin_memory()
        self.hout = torch.empty((self.pool_rows, N), dtype=torch.bfloat16).pin_memory()
        self.staging = torch.empty(2 * K * N * 2 + self.pool_rows * (K + N) * 2 + 4 * 256, dtype=torch.uint8, device="cuda")

    def run_step_e2e(self, stream):
        K, N = self.K, self.N
        h2d = d2h = 0
        for m in self.Ms:
            self.enc.encode(((m, K), (K, N), (K, N)))
            code = self.dvm.Code(self.enc.buf, self.enc.size.value, None)
            self.dvm.run_host(code, [self.hx[:m], self.hwg, self.hwu, self.hout[:m]], self.staging, stream)
            h2d += 2 * K * N * 2 + m * K * 2
            d2h += m * N * 2
        return h2d, d2h

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        K, N = self.K, self.N
        wg, wu = wl.to_f64(self.wg), wl.to_f64(self.wu)
        t_all, flops, rows_done, off, m = 0.0, 0, 0, 0, min(256, self.pool_rows)
        while t_all < budget_s:
            if off + m > self.pool_rows:
                off = 0
            x = wl.to_f64(self.x[off:off + m])
            t0 = time.perf_counter(); orc.evaluate(self.prog.nodes, [x, wg, wu]); t_all += time.perf_counter() - t0
            flops += 4 * m * K * N
            rows_done += m; off += m
        return flops / t_all / 1e12, t_all, f"{rows_done} rows of X in windows of {m} rows against both full weight matrices, numpy float64"


class AddmmWorkload:
    """addmm over the paper's LLM (n,k) pairs (Table 2): out = A[m,k] @ B[k,n] + C[m,n], bf16, fp32 accumulate."""
    name = "addmm"
    metric, unit, scale, bound, kernel, peak_key = "tflops_dynamic_shape_sweep", "TFLOP/s", 1e12, "tensor", "dvm_mm_kernel", "bf16_tflops_sustained"

    def __init__(self, dvm, n_instances=36, device="cuda", max_rows=0):
        self.dvm = dvm
        self.prog = wl.program_addmm()
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.shapes = wl.shapes_addmm(n_instances)
        if max_rows:
            self.shapes = [(min(m, max_rows), n, k) for m, n, k in self.shapes]
        seed = wl.data_seed("addmm", 0)
        self.B = {nk: wl.randn((nk[1], nk[0]), torch.bfloat16, seed + 10 + i, device, std=0.02)
                  for i, nk in enumerate(sorted({(n, k) for _, n, k in self.shapes}))}   # weights: once per (n, k)
        mmax = max(m for m, _, _ in self.shapes)
        kmax = max(k for _, _, k in self.shapes); nmax = max(n for _, n, _ in self.shapes)
        self.a_pool = wl.randn((mmax * kmax,), torch.bfloat16, seed, device)
        self.c_pool = wl.randn((mmax * nmax,), torch.bfloat16, seed + 1, device)
        self.o_pool = torch.empty((mmax * nmax,), dtype=torch.bfloat16, device=device)
        self.work_per_instance = [2 * m * n * k for m, n, k in self.shapes]
        self.bytes_per_instance = [2 * (m * k + k * n + 2 * m * n) for m, n, k in self.shapes]
        self.total_work = sum(self.work_per_instance)
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = (f"addmm: A[m,k] @ B[k,n] + C[m,n], bf16, fp32 accumulate, bf16 out; {n_instances} dynamic instances, "
                            "m 1..8192, (n,k) cycling through the nine LLM pairs of the paper's Table 2, each re-encoded per launch")
        self.l2_policy = "every instance streams its weight matrix (33..470 MB) and its own A / C / out windows"

    def _args(self, i):
        import ctypes as C
        m, n, k = self.shapes[i]
        return (C.c_void_p * 4)(self.a_pool.data_ptr(), self.B[(n, k)].data_ptr(), self.c_pool.data_ptr(), self.o_pool.data_ptr())

    def run_step(self, stream, events=None, enc_ns=None):
        lib_launch = self.dvm.binding.lib.dvm_launch
        for i, (m, n, k) in enumerate(self.shapes):
            t0 = time.perf_counter_ns()
            size = self.enc.encode(((m, k), (k, n), (m, n)))
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            arr = self._args(i)
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(self.enc.buf, size, arr, 4, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.shapes)

    def setup_e2e(self):
        self.staging = None   # the weights alone are 1.6 GB per sweep over PCIe: no end-to-end leg for this workload

    def run_step_e2e(self, stream):
        return None

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        n, k = 4096, 4096
        b = wl.to_f64(self.B[(n, k)]) if (n, k) in self.B else wl.to_f64(wl.randn((k, n), torch.bfloat16, 1, std=0.02))
        t_all, flops, m = 0.0, 0, 256
        while t_all < budget_s:
            a = wl.to_f64(self.a_pool[:m * k]).reshape(m, k); c = wl.to_f64(self.c_pool[:m * n]).reshape(m, n)
            t0 = time.perf_counter(); orc.evaluate(self.prog.nodes, [a, b, c]); t_all += time.perf_counter() - t0
            flops += 2 * m * n * k
        return flops / t_all / 1e12, t_all, f"[256,4096] @ [4096,4096] + [256,4096] repeated for {t_all:.0f} s, numpy float64"


class IfElseWorkload:
    """The paper's if-else-add compound operator (a > b ? 2x : 4x) + y, fp32 [b,s,f] (Table 2), dynamic instances."""
    name = "ifelse"

    def __init__(self, dvm, n_instances=50, device="cuda"):
        self.dvm = dvm
        self.prog = wl.program_if_else_add()
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.shapes = wl.shapes_if_else_add(n_instances)
        self.elems = [b * s_ * f for b, s_, f in self.shapes]
        self.pool = max(self.elems)
        seed = wl.data_seed("ifelse", 0)
        self.ins = [wl.randn((self.pool,), torch.float32, seed + i, device) for i in range(4)]
        self.out = torch.empty((self.pool,), dtype=torch.float32, device=device)
        self.bytes_per_instance = [20 * n for n in self.elems]   # four fp32 reads, one fp32 write per element
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = ("ifelse: (a > b ? 2x : 4x) + y, fp32 [b,s,f], b 1..256, s 1..512, f 1..8192 (instances above "
                            f"2^27 elements redrawn), {n_instances} dynamic instances, each re-encoded per launch")
        self.l2_policy = "mean instance 0.8 GB over five tensors, far above L2"

    def run_step(self, stream, events=None, enc_ns=None):
        import ctypes as C
        lib_launch = self.dvm.binding.lib.dvm_launch
        arr = (C.c_void_p * 5)(*[t.data_ptr() for t in self.ins], self.out.data_ptr())
        for shp in self.shapes:
            t0 = time.perf_counter_ns()
            size = self.enc.encode((shp,) * 4)
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(self.enc.buf, size, arr, 5, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.shapes)

    def setup_e2e(self):
        self.staging = None

    def run_step_e2e(self, stream):
        return None

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        n = 1 << 22
        ins = [wl.to_f64(t[:n]).reshape(1, 512, 8192) for t in self.ins]
        t_all, k = 0.0, 0
        while t_all < budget_s:
            t0 = time.perf_counter(); orc.evaluate(self.prog.nodes, ins); t_all += time.perf_counter() - t0; k += 1
        return k * 20 * n / t_all / 1e9, t_all, f"{k} evaluations of a [1,512,8192] instance, numpy float64"


class ViewsWorkload:
    """Views (Table 1, ViewLoad): out = 0.5 * x + y on bf16 [B,32,S,128], x read through a head-transpose view of
    storage laid out [B,S,32,128], dynamic (B, S) instances."""
    name = "views"
    H, D = 32, 128

    def __init__(self, dvm, n_instances=60, device="cuda"):
        self.dvm = dvm
        self.prog = wl.program_head_transpose_add()
        self.p = dvm.program_from_nodes(self.prog.nodes)
        self.enc = dvm.binding.Encoder(self.p)
        self.shapes = wl.shapes_views(n_instances, self.H, self.D)
        self.elems = [b * s_ * self.H * self.D for b, s_ in self.shapes]
        self.pool = max(self.elems)
        seed = wl.data_seed("views", 0)
        self.ins = [wl.randn((self.pool,), torch.bfloat16, seed + i, device) for i in range(2)]
        self.out = torch.empty((self.pool,), dtype=torch.bfloat16, device=device)
        self.bytes_per_instance = [6 * n for n in self.elems]   # two bf16 reads, one bf16 write per element
        self.total_bytes = sum(self.bytes_per_instance)
        self.description = ("views: out = 0.5*x + y, bf16 [B,32,S,128], x a head-transpose VIEW of [B,S,32,128] storage "
                            f"(rows of 128 elements, 256 B apart in groups), B 1..32, S 1..8192, {n_instances} dynamic "
                            "instances, each re-encoded per launch (dvm_encode_strided)")
        self.l2_policy = "mean instance 0.7 GB over three tensors, far above L2"

    def _strides(self, b, s_):
        H, D = self.H, self.D
        return [[s_ * H * D, D, H * D, 1], None]   # element (b,h,s,d) of x lies at ((b*S + s)*H + h)*D + d

    def run_step(self, stream, events=None, enc_ns=None):
        import ctypes as C
        lib_launch = self.dvm.binding.lib.dvm_launch
        arr = (C.c_void_p * 3)(*[t.data_ptr() for t in self.ins], self.out.data_ptr())
        for b, s_ in self.shapes:
            shp = (b, self.H, s_, self.D)
            t0 = time.perf_counter_ns()
            size = self.enc.encode((shp, shp), (), self._strides(b, s_))
            t1 = time.perf_counter_ns()
            if enc_ns is not None:
                enc_ns.append(t1 - t0)
            if events is not None:
                e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
                e0.record(stream)
            st = lib_launch(self.enc.buf, size, arr, 3, stream.cuda_stream)
            if st != 0:
                raise self.dvm.DvmError(st, "dvm_launch")
            if events is not None:
                e1.record(stream)
                events.append((e0, e1))
        return len(self.shapes)

    def setup_e2e(self):
        self.staging = None

    def run_step_e2e(self, stream):
        return None

    def oracle_sample(self, budget_s=12.0):
        from oracle import dvm_oracle as orc
        B, S = 2, 512
        n = B * S * self.H * self.D
        x = wl.to_f64(self.ins[0][:n])
        y = wl.to_f64(self.ins[1][:n]).reshape(B, self.H, S, self.D)
        t_all, k = 0.0, 0
        while t_all < budget_s:
            t0 = time.perf_counter()
            xv = orc.view_load(x, 0, (B, self.H, S, self.D), (S * self.H * self.D, self.D, self.H * self.D, 1))
            orc.evaluate(self.prog.nodes, [xv, y])
            t_all += time.perf_counter() - t0; k += 1
        return k * 6 * n / t_all / 1e9, t_all, f"{k} evaluations of a [2,32,512,128] instance (view_load + program), numpy float64"


WORKLOADS = {"views": ViewsWorkload, "ifelse": IfElseWorkload, "addmm": AddmmWorkload, "c1": C1Workload, "c2": C2Workload, "c3": C3Workload, "c4": C4Workload, "c5": C5Workload}
for _W in (C1Workload, C2Workload, C3Workload, C4Workload, IfElseWorkload, ViewsWorkload):   # the memory-bound sweeps: work = algorithmic bytes
    _W.metric, _W.unit, _W.scale, _W.bound = "hbm_gbs_dynamic_shape_sweep", "GB/s", 1e9, "hbm"
    _W.kernel, _W.peak_key = "dvm_vm_kernel", "hbm_gbs"
for _W in (C1Workload, C2Workload, C3Workload, IfElseWorkload, ViewsWorkload):   # one program per launch that the lean interpreter runs
    _W.kernel = "dvm_vm_lean_kernel"


def oracle_threads(workload: str) -> int:
    """Threads the numpy oracle actually uses: elementwise programs run on one core; the matmul of c5 goes
    through numpy's BLAS, which uses its own pool."""
    if workload not in ("c5", "addmm"):
        return 1
    try:
        from threadpoolctl import threadpool_info
        n = [d.get("num_threads", 1) for d in threadpool_info() if d.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return 1



# ----------------------------------------------------------------------------- oracle spot checks (cpu_baseline leg)
def _check_cases(name):
    """Small seeded cases of a workload's program(s): (program, cpu inputs, runtime scalars, input strides or None)."""
    bf = torch.bfloat16
    if name == "c1":
        return [(wl.program_c1(), wl.inputs_c1(), (), None)]
    if name == "c2":
        return [(wl.program_add_rmsnorm(4096), wl.inputs_add_rmsnorm(333, 4096, 1), (), None)]
    if name == "c3":
        return [(wl.program_masked_softmax(), wl.inputs_masked_softmax(1, 2, 333, 2), (), None),
                (wl.program_masked_softmax(), wl.inputs_masked_softmax(1, 1, 1024, 3), (), None)]
    if name == "c4":
        out = []
        for j, (kind, r, c) in enumerate([("gelu_affine", 200, 333), ("layernorm", 17, 1000), ("sigmoid_mul", 64, 4095)]):
            ins, params = wl.inputs_stack(kind, r, c, 40 + 4 * j)
            out.append((wl.stack_program(kind), ins, params, None))
        return out
    if name == "c5":
        return [(wl.program_mlp_gate(), [wl.randn((96, 512), bf, 3), wl.randn((512, 1024), bf, 4, std=0.05),
                                         wl.randn((512, 1024), bf, 5, std=0.05)], (), None)]
    if name == "addmm":
        return [(wl.program_addmm(), [wl.randn((130, 512), bf, 6), wl.randn((512, 520), bf, 7, std=0.05),
                                      wl.randn((130, 520), bf, 8)], (), None)]
    if name == "ifelse":
        return [(wl.program_if_else_add(), [wl.randn((3, 50, 333), torch.float32, 10 + i) for i in range(4)], (), None)]
    if name == "views":
        B, H, S, D = 2, 32, 100, 128
        xs = wl.randn((B * S * H * D,), bf, 20)
        y = wl.randn((B, H, S, D), bf, 21)
        return [(wl.program_head_transpose_add(), [xs, y], (), [[S * H * D, D, H * D, 1], None], (B, H, S, D))]
    return []


def oracle_check(dvm, name):
    """Runs the workload's small cases through the C ABI on the GPU and through the CPU oracle, element by element:
    worst row-scaled error |g - o| / max(|o|, row max |o|) against the gate (1e-5 fp32 programs, 2e-2 programs with a
    bf16 tensor), and the strict elementwise statistics for the programs that only the row-scaled gate can hold."""
    import numpy as np
    from oracle import dvm_oracle as orc
    worst, n_el, ok = 0.0, 0, True
    strict = {"max": 0.0, "n_over": 0, "n_well": 0, "n_over_well": 0, "n": 0}
    gate = 1e-5
    stacked = name == "c4"
    codes, tls, wants, progs_seen = [], [], [], []
    if stacked:
        dvm.set_elems_per_thread(32)
    try:
        for case in _check_cases(name):
            prog, ins, params, strides = case[:4]
            kinds = [n[1] for n in prog.nodes if n[0] == "input"] + [n[2] for n in prog.nodes if n[0] == "output"]
            r = 2e-2 if "bf16" in kinds else 1e-5
            gate = max(gate, r) if r == 2e-2 else gate
            dev = [t.cuda() for t in ins]
            shapes = [tuple(t.shape) for t in ins]
            ins64 = [wl.to_f64(t) for t in ins]
            if strides is not None:   # the first input is storage seen through a view
                shapes[0] = case[4]
                ins64[0] = orc.view_load(ins64[0], 0, case[4], strides[0])
                code = dvm.encode(dvm.program_from_nodes(prog.nodes), shapes, params, in_strides=strides)
            else:
                code = dvm.encode(dvm.program_from_nodes(prog.nodes), shapes, params)
            dt = {"f32": torch.float32, "bf16": torch.bfloat16}
            outs = [torch.full(sh, float("nan"), dtype=dt[nd[2]], device="cuda") for sh, nd in zip(code.out_shapes, prog.output_nodes)]
            want = orc.evaluate(prog.nodes, ins64, params)
            want32 = orc.evaluate(prog.nodes, ins64, params, diagnostic_fp32=True)
            if stacked:
                codes.append(code); tls.append(dev + outs)
            else:
                dvm.launch(code, dev + outs)
            wants.append((outs, want, want32, r))
        if stacked:
            dvm.launch_stacked(codes, tls)
        assert dvm.last_device_status() == 0
        for outs, want, want32, r in wants:
            for g, w, w32 in zip(outs, want, want32):
                g = wl.to_f64(g)
                den = np.maximum(np.abs(w), np.max(np.abs(w), axis=-1, keepdims=True))
                err = np.abs(g - w)
                bad = ~(err <= r * den)
                ok = ok and not bool(bad.any())
                with np.errstate(divide="ignore", invalid="ignore"):
                    g1 = np.where(err == 0, 0.0, err / den)
                    rel = np.where((w != 0) & np.isfinite(w), err / np.abs(w), 0.0)
                worst = max(worst, float(np.nanmax(g1)) if g1.size else 0.0)
                well = (w != 0) & (np.abs(w32 - w) <= 1e-6 * np.abs(w))
                over = rel > r
                strict["max"] = max(strict["max"], float(rel.max()) if rel.size else 0.0)
                strict["n_over"] += int(over.sum()); strict["n_well"] += int(well.sum())
                strict["n_over_well"] += int((over & well).sum()); strict["n"] += int(w.size)
                n_el += int(w.size)
    finally:
        if stacked:
            dvm.set_elems_per_thread(0)
    return {"pass": bool(ok), "worst_g1": worst, "gate": gate, "elements": n_el,
            "strict": {"max": strict["max"], "n_over_gate": strict["n_over"], "n_well_conditioned": strict["n_well"],
                       "n_over_gate_well_conditioned": strict["n_over_well"], "n": strict["n"],
                       "note": "strict |g-o|/|o| (reported, not gated); well conditioned = a faithful fp32 evaluation is within 1e-6 of the fp64 oracle"}}


def native_encode_us(W, reps):
    """Host encode latency measured inside the library (steady clock around the encoder, no binding): `reps` repeats of
    each of up to 20 instances of the sweep."""
    import numpy as np
    if not hasattr(W, "enc"):
        return None
    if W.name == "views":
        cases = [(((b, W.H, s_, W.D),) * 2, (), W._strides(b, s_)) for b, s_ in W.shapes[:20]]
    elif W.name == "ifelse":
        cases = [((shp,) * 4, (), None) for shp in W.shapes[:20]]
    elif W.name == "addmm":
        cases = [(((m, k), (k, n), (m, n)), (), None) for m, n, k in W.shapes[:20]]
    elif W.name == "c1":
        cases = [(((7, 1531),) * 3, (), None)]
    elif W.name == "c2":
        cases = [(((t, 4096), (t, 4096), (4096,)), (), None) for t in W.rows[:20]]
    elif W.name == "c3":
        cases = [(((b, 32, s_, s_), (1, 1, s_, s_)), (), None) for b, s_ in W.shapes[:20]]
    elif W.name == "c5":
        cases = [(((m, 4096), (4096, 11008), (4096, 11008)), (), None) for m in W.Ms[:20]]
    else:
        return None
    ns = []
    for shp, sc, strides in cases:
        ns += W.enc.time_encode(shp, sc, reps, strides)
    a = np.sort(np.asarray(ns, dtype=np.float64)) / 1e3
    return {"mean": float(a.mean()), "p50": float(a[len(a) // 2]), "p99": float(a[int(0.99 * len(a))]),
            "p999": float(a[int(0.999 * len(a))]), "max": float(a[-1]), "n": int(len(a)),
            "note": f"steady clock inside the library around the encoder, {reps} repeats of each of {len(cases)} instances"}


def run_config(dvm, name, peaks, peak_kind, steps, warmup=3, check=True, baseline_s=1.5):
    """One sweep of another workload for the `configs` object of the default line: kernel-only throughput over `steps`
    timed steps after `warmup`, roofline fraction, host encode latency, and the oracle beside it (throughput on a
    bounded sample, spot check of small cases)."""
    import gc
    kw = {}
    W = WORKLOADS[name](dvm, **kw)
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        W.run_step(stream)
    torch.cuda.synchronize()
    events, enc_ns = [], []
    gc_was = gc.isenabled()
    gc.disable()
    try:
        l0 = dvm.launch_count()
        e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            W.run_step(stream, events=events, enc_ns=enc_ns)
        e1.record(stream)
        torch.cuda.synchronize()
        launches = dvm.launch_count() - l0
    finally:
        if gc_was:
            gc.enable()
    assert dvm.last_device_status() == 0
    ms = e0.elapsed_time(e1) / steps
    work_each = getattr(W, "work_per_instance", W.bytes_per_instance)
    value = sum(work_each) / (ms * 1e-3) / W.scale
    kern_ms = [a.elapsed_time(b) for a, b in events]
    achieved = sum(work_each) * steps / (sum(kern_ms) * 1e-3) / W.scale
    peak = peaks[W.peak_key]
    enc_us = sorted(x / 1e3 for x in enc_ns)
    out = {"workload": W.description, "value": value, "unit": W.unit, "ms_per_step": ms, "steps": steps, "warmup": warmup,
           "roofline": {"bound": W.bound, "achieved": achieved, "peak": peak, "frac": achieved / peak,
                        "peak_kind": f"of {peak_kind} ({W.peak_key})",
                        "frac_of_nominal": achieved / (2250.0 if W.bound == "tensor" else 8000.0)},
           "launches_timed": len(kern_ms), "gpu_launches": launches,
           "encode_us": {"mean": sum(enc_us) / len(enc_us), "p99": enc_us[min(len(enc_us) - 1, int(0.99 * len(enc_us)))],
                         "max": enc_us[-1], "n": len(enc_us),
                         "note": ("per program, one dvm_encode_batch call of 64 programs" if name == "c4" else
                                  "perf_counter around the binding's encode call, garbage collector off")},
           "encode_us_native": native_encode_us(W, 200)}
    if name == "c1":
        out["latency_us"] = {"kernel_event_mean": 1e3 * sum(kern_ms) / max(len(kern_ms), 1)}
    if check:
        v, dt, sample = W.oracle_sample(budget_s=baseline_s)
        out["cpu_baseline"] = {"value": v, "unit": W.unit, "cores": getattr(W, "oracle_cores", None) or oracle_threads(name), "kind": "oracle", "sample": sample,
                               "seconds": dt, "check": oracle_check(dvm, name)}
    del W
    torch.cuda.empty_cache()
    # a workload may have set the encoder's knobs for its own programs (c4): the next one starts from the defaults
    dvm.set_elems_per_thread(0)
    dvm.set_min_resident_ctas(0)
    dvm.set_stacked_one_slot(False)
    return out


# ----------------------------------------------------------------------------- reference arm
def run_reference(args):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import dvm_oracle as orc
    if args.workload == "c2":
        prog = wl.program_add_rmsnorm(4096)
        rows = 4096
        seed = wl.data_seed("c2", 0)
        ins = [wl.to_f64(t) for t in wl.inputs_add_rmsnorm(rows, 4096, seed)]
        nbytes = rows * 4096 * 8 + 8192
        sample = f"{rows} rows x 4096 (one c2 instance) per step, numpy float64"
        desc = C2Workload.__doc__
        params = ()
    elif args.workload == "ifelse":
        prog = wl.program_if_else_add()
        ins = [wl.to_f64(wl.randn((1, 512, 8192), torch.float32, 1 + i)) for i in range(4)]
        nbytes = 20 * 512 * 8192
        sample = "one [1,512,8192] instance per step, numpy float64"
        desc = IfElseWorkload.__doc__
        params = ()
    elif args.workload == "views":
        prog = wl.program_head_transpose_add()
        B, S, H, D = 2, 512, 32, 128
        xs = wl.to_f64(wl.randn((B * S * H * D,), torch.bfloat16, 1))
        ins = [orc.view_load(xs, 0, (B, H, S, D), (S * H * D, D, H * D, 1)), wl.to_f64(wl.randn((B, H, S, D), torch.bfloat16, 2))]
        nbytes = 6 * B * S * H * D
        sample = "one [2,32,512,128] instance per step (program on the loaded view), numpy float64"
        desc = ViewsWorkload.__doc__
        params = ()
    elif args.workload == "addmm":
        prog = wl.program_addmm()
        M = 128
        ins = [wl.to_f64(wl.randn((M, 4096), torch.bfloat16, 1)), wl.to_f64(wl.randn((4096, 4096), torch.bfloat16, 2, std=0.02)),
               wl.to_f64(wl.randn((M, 4096), torch.bfloat16, 3))]
        nbytes = 2 * M * 4096 * 4096   # flops
        sample = f"[{M},4096] @ [4096,4096] + [{M},4096] per step, numpy float64"
        desc = AddmmWorkload.__doc__
        params = ()
    elif args.workload == "c1":
        prog = wl.program_c1()
        ins = [wl.to_f64(t) for t in wl.inputs_c1()]
        nbytes = 16 * 7 * 1531
        sample = "the [7,1531] instance per step, numpy float64"
        desc = C1Workload.__doc__
        params = ()
    elif args.workload == "c3":
        prog = wl.program_masked_softmax(128)
        ins = [wl.to_f64(t) for t in wl.inputs_masked_softmax(1, 8, 512, wl.data_seed("c3", 0))]
        nbytes = 8 * 512 * 512 * 4 + 2 * 512 * 512
        sample = "scores [1,8,512,512] per step, numpy float64"
        desc = C3Workload.__doc__
        params = ()
    elif args.workload == "c5":
        prog = wl.program_mlp_gate()
        M = 64
        ins = [wl.to_f64(t) for t in wl.inputs_mlp_gate(M, 4096, 11008, wl.data_seed("c5", 0))]
        nbytes = 4 * M * 4096 * 11008   # flops
        sample = f"X [{M},4096] against both weight matrices per step, numpy float64"
        desc = C5Workload.__doc__
        params = ()
    else:
        prog = wl.program_sigmoid_mul()
        ins = [wl.to_f64(t) for t in wl.inputs_stack("sigmoid_mul", 512, 4096, 1)[0]]
        nbytes = 12 * 512 * 4096
        sample = "one sigmoid(x)*y program [512,4096] per step, numpy float64"
        desc = C4Workload.__doc__
        params = ()
    tensor = args.workload in ("c5", "addmm")
    cores = oracle_threads(args.workload)
    if tensor:   # the matmul goes through numpy's BLAS, which uses the host cores itself
        for _ in range(args.warmup):
            orc.evaluate(prog.nodes, ins, params)
        t0 = time.perf_counter()
        for _ in range(args.steps):
            orc.evaluate(prog.nodes, ins, params)
        dt = time.perf_counter() - t0
    else:        # elementwise programs: one worker process per host core, each evaluates the sample once per step
        from oracle import parallel as opar
        pool = opar.StepPool(prog.nodes, [ins], params)
        cores = pool.n
        for _ in range(args.warmup):
            pool.step()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            pool.step()
        dt = time.perf_counter() - t0
        pool.close()
        nbytes *= cores
        sample += f", evaluated once per step by each of {cores} worker processes (one per host core)"
    val = nbytes * args.steps / dt / (1e12 if tensor else 1e9)
    unit = "TFLOP/s" if tensor else "GB/s"
    line = {"impl": "reference", "metric": "tflops_dynamic_shape_sweep" if tensor else "hbm_gbs_dynamic_shape_sweep",
            "value": val, "unit": unit,
            "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": desc, "sample": sample},
            "cpu_baseline": {"value": val, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def encode_latency(W, reps):
    """Host encode latency over `reps` repeats of each of (up to) 20 instances of the sweep: pure dvm_encode calls."""
    if W.name == "views":
        ns = []
        for b, s_ in W.shapes[:20]:
            shp = (b, W.H, s_, W.D)
            for _ in range(reps):
                t0 = time.perf_counter_ns(); W.enc.encode((shp, shp), (), W._strides(b, s_)); ns.append(time.perf_counter_ns() - t0)
        us = sorted(x / 1e3 for x in ns)
        return {"mean": sum(us) / len(us), "p50": us[len(us) // 2], "p99": us[int(0.99 * len(us))], "max": us[-1],
                "n": len(us), "note": f"{reps} repeats of each of 20 instances, perf_counter around the binding's dvm_encode_strided call"}
    if W.name == "ifelse":
        shapes = [(shp,) * 4 for shp in W.shapes[:20]]
    elif W.name == "addmm":
        shapes = [((m, k), (k, n), (m, n)) for m, n, k in W.shapes[:20]]
    elif W.name == "c1":
        shapes = [((7, 1531),) * 3]
    elif W.name == "c2":
        shapes = [((t, 4096), (t, 4096), (4096,)) for t in W.rows[:20]]
    elif W.name == "c3":
        shapes = [((b, 32, s_, s_), (1, 1, s_, s_)) for b, s_ in W.shapes[:20]]
    else:
        shapes = [((m, 4096), (4096, 11008), (4096, 11008)) for m in W.Ms[:20]]
    ns = []
    for shp in shapes:
        for _ in range(reps):
            t0 = time.perf_counter_ns(); W.enc.encode(shp); ns.append(time.perf_counter_ns() - t0)
    us = sorted(x / 1e3 for x in ns)
    return {"mean": sum(us) / len(us), "p50": us[len(us) // 2], "p99": us[int(0.99 * len(us))], "max": us[-1],
            "n": len(us), "note": f"{reps} repeats of each of {len(shapes)} instances, perf_counter around the ctypes call"}


# ----------------------------------------------------------------------------- multi-rank aggregation
def reduce_max_over_ranks(x: float, dist, device) -> float:
    """The slowest rank's time: all-reduce MAX over the process group (identity without one)."""
    t = torch.tensor([x], dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(work_per_rank: float, world: int, ms_per_step: float, scale: float) -> float:
    """Replicas only: every rank processes the same sweep, the job's work is world x one rank's."""
    return work_per_rank * world / (ms_per_step * 1e-3) / scale


# ----------------------------------------------------------------------------- main arm
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None,
                    help="timed passes over the sweep (default 5; 100 for the matmul workloads, about two seconds: their "
                         "roofline is the SUSTAINED cuBLAS rate under the power cap, which a 0.1 s run does not meet)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="c2", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="dvm", choices=["dvm", "reference"])
    ap.add_argument("--instances", type=int, default=0, help="override the number of instances (debug)")
    ap.add_argument("--max-rows", type=int, default=0, help="cap rows per instance (small profiling case)")
    ap.add_argument("--elems-per-thread", type=int, default=0, help="fix the encoder's elements per thread (16/32/64; 0 = cost model)")
    ap.add_argument("--encode-reps", type=int, default=1000, help="repeats per instance of the host-encode latency measurement")
    ap.add_argument("--general-interpreter", action="store_true",
                    help="run every launch on the general interpreter instead of the lean one (for comparisons)")
    ap.add_argument("--lean-stacked", action="store_true",
                    help="run stacked launches on the lean interpreter too (default: the general one; for comparisons)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-configs", action="store_true",
                    help="skip the sweeps of the other workloads that the default line reports under `configs`")
    ap.add_argument("--detail", default="", help="write per-instance timings to this JSON file")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.steps is None:
            args.steps = 5
        return run_reference(args)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the DVM path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
        dist = dist_mod

    import paper_2603_24239_b200 as dvm
    from paper_2603_24239_b200 import binding
    dvm.binding = binding

    kw = {}
    if args.elems_per_thread:
        dvm.set_elems_per_thread(args.elems_per_thread)
    if args.general_interpreter:
        dvm.set_lean_kernel(False)
    if args.lean_stacked:
        dvm.set_lean_kernel(2)
    if args.instances:
        kw = {"n_launches": args.instances} if args.workload == "c4" else {"n_instances": args.instances}
    if args.max_rows and args.workload in ("c2", "c5", "addmm"):
        kw["max_rows"] = args.max_rows
    W = WORKLOADS[args.workload](dvm, **kw)
    if args.steps is None:
        args.steps = 100 if W.bound == "tensor" else 5
    stream = torch.cuda.current_stream()
    peaks, peak_kind = measured_peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        W.run_step(stream)
    barrier()
    assert dvm.last_device_status() == 0

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    launches0 = dvm.launch_count()
    events, enc_ns = [], []
    step_ms = []
    barrier()
    e_start = torch.cuda.Event(enable_timing=True); e_end = torch.cuda.Event(enable_timing=True)
    import gc
    gc.collect()
    gc.disable()   # a collection inside the sweep would show up as a host-encode outlier of a millisecond
    e_start.record(stream)
    n_inst = 0
    for k in range(args.steps):
        n_inst = W.run_step(stream, events=events, enc_ns=enc_ns)
    e_end.record(stream)
    gc.enable()
    barrier()
    total_ms = e_start.elapsed_time(e_end)
    launches = dvm.launch_count() - launches0
    clocks = sampler.stop() if rank == 0 else None
    assert dvm.last_device_status() == 0

    total_ms = reduce_max_over_ranks(total_ms, dist, "cuda")
    ms_per_step = total_ms / args.steps
    work_each = getattr(W, "work_per_instance", W.bytes_per_instance)
    total_work = sum(work_each)
    value = whole_job_value(total_work, world, ms_per_step, W.scale)

    # dominant kernel: algorithmic bytes per launch over its CUDA-event time
    kern_ms = [a.elapsed_time(b) for a, b in events]
    per_launch_bytes = W.bytes_per_instance * args.steps
    per_launch_work = work_each * args.steps
    kernel_total_ms = sum(kern_ms)
    achieved = sum(per_launch_work) / (kernel_total_ms * 1e-3) / W.scale
    peak = peaks[W.peak_key]
    if W.bound == "hbm":   # "large shapes": instances moving >= 256 MB
        big = [(b, m) for b, m in zip(per_launch_work, kern_ms) if b >= 256e6]
    else:                  # instances that are tensor-bound by a wide margin (M >= 1024)
        big = [(b, m) for b, m in zip(per_launch_work, kern_ms) if b >= 4 * 1024 * 4096 * 11008 / (2 if W.name == "addmm" else 1)]
    large_gbs = (sum(b for b, _ in big) / (sum(m for _, m in big) * 1e-3) / W.scale) if big else None
    gbs_each = sorted(b / (m * 1e-3) / W.scale for b, m in zip(per_launch_work, kern_ms))
    # per-launch roofline time: the slower of (flops / tensor peak) and (bytes / HBM peak)
    roof_ms = [max((w / (peak * 1e12) if W.bound == "tensor" else 0.0), b / (peaks["hbm_gbs"] * 1e9)) * 1e3
               for w, b in zip(per_launch_work, per_launch_bytes)]
    roofline_time_frac = sum(roof_ms) / kernel_total_ms
    enc_us = sorted(x / 1e3 for x in enc_ns)

    def pct(v, q):
        return v[min(len(v) - 1, int(q * len(v)))] if v else None

    traffic = None
    tp = os.path.join(ROOT, "profiles", f"{W.kernel}_{args.workload}.md")
    if os.path.exists(tp):
        import re
        mt = re.search(r"dram_bytes_per_algorithmic_byte:\s*([0-9.]+)", open(tp).read())
        if mt:
            # measured DRAM bytes per algorithmic byte on an ncu-captured instance, scaled to the mean launch
            traffic = float(mt.group(1)) * sum(per_launch_bytes) / len(per_launch_bytes)
    traffic_source = (f"ratio DRAM bytes / algorithmic bytes of the ncu capture summarised in profiles/{W.kernel}_{args.workload}.md "
                      "(a committed measurement of a smaller instance, not taken in this run), scaled to the mean launch") if traffic else None

    line = {
        "metric": W.metric, "value": value, "unit": W.unit, "n_gpus": world,
        "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 x bf16 -> f32" if W.bound == "tensor" else "f32", "data": "synthetic",
        "config": {"workload": W.description, "l2": W.l2_policy, "instances_per_step": n_inst,
                   "algorithmic_bytes_per_step": W.total_bytes,
                   "algorithmic_flops_per_step": total_work if W.bound == "tensor" else None,
                   "multi_gpu": "replicas only (no collective)"},
        "pct_of_nominal": {"value": value / world / (2250.0 if W.bound == "tensor" else 8000.0),
                           "nominal": "2.25 PFLOP/s dense bf16" if W.bound == "tensor" else "8 TB/s"},
        "encode_us": {"mean": sum(enc_us) / len(enc_us), "p50": pct(enc_us, 0.5), "p99": pct(enc_us, 0.99),
                      "max": enc_us[-1], "n": len(enc_us), "note": ("per program: perf_counter around one dvm_encode_batch call of 64 programs, argument marshalling included"
                               if W.name == "c4" else "perf_counter around the ctypes call to dvm_encode")},
        "roofline": {"bound": W.bound, "kernel": W.kernel, "achieved": achieved, "peak": peak,
                     "unit": W.unit, "frac": achieved / peak, "peak_kind": f"of {peak_kind} ({W.peak_key})",
                     "traffic": traffic, "traffic_source": traffic_source, "large_instances": large_gbs,
                     "large_instances_frac": (large_gbs / peak) if large_gbs else None,
                     "roofline_time_frac": roofline_time_frac,
                     "per_launch": {"min": gbs_each[0], "p10": pct(gbs_each, 0.1), "p50": pct(gbs_each, 0.5),
                                    "max": gbs_each[-1]},
                     "launches_timed": len(kern_ms), "kernel_ms_per_step": kernel_total_ms / args.steps},
        "gpu_launches": launches,
        "clocks": clocks,
    }
    if rank == 0 and W.name == "c1":
        # the figure of merit of the latency-bound config: host wall time of encode + launch + sync, and the
        # device time between events around the launch
        wall = []
        for _ in range(300):
            t0 = time.perf_counter_ns(); W.run_step(stream); stream.synchronize(); wall.append((time.perf_counter_ns() - t0) / 1e3)
        wall.sort()
        line["latency_us"] = {"encode_launch_sync_wall_p50": wall[len(wall) // 2], "wall_p99": wall[int(0.99 * len(wall))],
                              "kernel_event_mean": 1e3 * kernel_total_ms / max(len(kern_ms), 1)}
    if rank == 0 and hasattr(W, "enc") and args.encode_reps > 0:
        line["encode_us_repeated"] = encode_latency(W, args.encode_reps)
        line["encode_us_native"] = native_encode_us(W, args.encode_reps)
    if args.detail and rank == 0:
        with open(args.detail, "w") as f:
            json.dump({"bytes": per_launch_bytes, "ms": kern_ms, "enc_us": [x / 1e3 for x in enc_ns]}, f)

    # ---- end to end through dvm_run_host with pinned host buffers (copies inside the timed region) ----
    e2e = None
    if not args.no_e2e:
        W.setup_e2e()
        if getattr(W, "staging", None) is not None:
            barrier()
            t0 = time.perf_counter()
            h2d, d2h = W.run_step_e2e(stream)
            torch.cuda.synchronize()
            dt = time.perf_counter() - t0
            dt = reduce_max_over_ranks(dt, dist, "cuda")
            e2e_work = getattr(W, "e2e_work", total_work)   # c4 runs its first launches only
            e2e = {"value": whole_job_value(e2e_work, world, dt * 1e3, W.scale), "unit": W.unit,
                   "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": 1,
                   "note": ("first %d launches: pinned host -> device, dvm_launch_stacked, device -> pinned host, sync"
                            % W.E2E_LAUNCHES) if W.name == "c4" else
                           "dvm_run_host per instance: pinned host -> device, launch, device -> pinned host, sync"}
    line["e2e"] = e2e

    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, dt, sample = W.oracle_sample()
        line["cpu_baseline"] = {"value": v, "unit": W.unit, "cores": getattr(W, "oracle_cores", None) or oracle_threads(W.name), "kind": "oracle",
                                "sample": sample, "seconds": dt, "host_cores_available": os.cpu_count(),
                                "check": oracle_check(dvm, W.name)}
    if rank == 0 and world == 1 and args.workload == "c2" and not args.no_configs and not args.instances and not args.max_rows:
        # the other sweeps, fewer steps each, so that every configuration is measured by the default command
        name_main = W.name
        del W
        torch.cuda.empty_cache()
        cfgs = {}
        # (the tensor-core sweeps first, while the GPU is coolest; c4 last: it changes the encoder's knobs)
        for name, steps in (("c5", 40), ("addmm", 40), ("ifelse", 2), ("views", 2), ("c1", 50), ("c3", 2), ("c4", 2)):
            if name == name_main:
                continue
            try:
                cfgs[name] = run_config(dvm, name, peaks, peak_kind, steps, check=not args.no_cpu_baseline)
            except Exception as e:   # one failing sweep must not take the headline line with it
                cfgs[name] = {"error": f"{type(e).__name__}: {e}"}
                torch.cuda.empty_cache()
        line["configs"] = cfgs
    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

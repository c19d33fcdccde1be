#!/usr/bin/env python
"""Benchmark of the hot path: whole-model Huffman decode + dequantisation to fp16.

A step is one pass of the whole path over one synthetic model: upload of the tensor
descriptors, construction of the per-tensor decode tables, and the persistent decode +
dequant kernel over every chunk of every tensor.  Default workload: mistral-7B-shaped
weights at uint8 (7.24e9 weights, 226 + 65 tensors); `--also uint4` adds the 4-bit run.

    python bench.py --gpus N --steps K --warmup W            # this library
    python bench.py --impl reference --gpus N ...            # the CPU oracle, host cores

One JSON line on stdout (rank 0).  Multi-GPU: every rank decodes its own full copy of the
model (no data-path collective; weak scaling), launched by torch.distributed.run.
"""
from __future__ import annotations

import argparse
import ctypes as C
import dataclasses
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

import workloads
from workloads.device import DeviceModel

METRIC = "Huffman decode+dequant GB/s (compressed in + fp16 out)"
NOMINAL_HBM_GBS = 8000.0
# DRAM bytes per weight of the decode kernel (dram__bytes_read.sum + dram__bytes_write.sum of one
# ncu capture on the 1-layer truncation, 480,260,096 weights; traffic grows in proportion to the
# weights, so a full launch is this figure times its weights).  See profiles/.  Set an entry to
# None when the kernel changes until the counters have been taken again.
NCU_DRAM_BYTES_PER_WEIGHT = {8: 1102.38e6 / 480260096, 4: 966.16e6 / 480260096}
FALLBACK_HBM_GBS = 6650.0


# ----------------------------------------------------------------------------- helpers

def measured_peak():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(p) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback (6.65 TB/s, earlier measurement on this pool)"


def pick_workload(name: str, max_layers):
    if name.endswith("-paperbits"):
        return workloads.with_paper_bit_rate(pick_workload(name[:-10], max_layers))
    if name.endswith("-gauss"):
        return workloads.with_matrix_kind(pick_workload(name[:-6], max_layers), "gauss")
    if name == "mistral8":
        return workloads.mistral_7b(bits=8, max_layers=max_layers)
    if name == "mistral4":
        return workloads.mistral_7b(bits=4, max_layers=max_layers)
    if name == "smollm8":
        return workloads.smollm_1p7b(max_layers=max_layers)
    if name == "phi3_4":
        return workloads.phi3_mini_4k(max_layers=max_layers)
    if name == "single":
        return workloads.single_tensor()
    raise SystemExit(f"unknown workload {name}")


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.005):
        super().__init__(daemon=True)
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.nv = None

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
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def stop(self):
        self._stop_evt.set()
        self.join(timeout=2)
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


# ----------------------------------------------------------------------------- this library

def time_steps(E, model, steps, warmup, world, sampler_index):
    import torch.distributed as dist
    for _ in range(warmup):
        E.entro_decode_dequant_batched(model.descs)
    torch.cuda.synchronize()
    assert E.entro_last_device_status() == E.OK
    E.entro_profile_begin(steps)
    launches0 = E.entro_kernel_launch_count()
    sampler = ClockSampler(sampler_index)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    for _ in range(steps):
        E.entro_decode_dequant_batched(model.descs)
    ev1.record()
    torch.cuda.synchronize()
    clocks = sampler.stop()
    if world > 1:
        dist.barrier()
    ms = ev0.elapsed_time(ev1)
    from paper_2505_02380_b200 import multirank
    ms = multirank.max_over_ranks(ms, "cuda")
    launches = E.entro_kernel_launch_count() - launches0
    kernel_ms = E.entro_profile_read(steps)
    E.entro_profile_begin(0)
    assert E.entro_last_device_status() == E.OK
    return ms, launches, kernel_ms, clocks


def time_symbols(E, model, steps=10):
    """The same model decoded to integer symbols (the paper's decoder output): one byte per
    symbol at 8 bits, two symbols per byte at 4 bits.  -> kernel ms, GB/s (compressed in + bytes out)."""
    packed = model.wl.bits == 4
    nbytes = [(t.numel + 1) // 2 if packed else t.numel for t in model.wl.tensors]
    buf = torch.empty(sum((b + 15) // 16 * 16 for b in nbytes), dtype=torch.uint8, device="cuda")
    descs, pos = [], 0
    for spec, enc, cb, nb in zip(model.wl.tensors, model.keep, model.cbs, nbytes):
        descs.append(E.make_desc_bytes(enc.stream, enc.index, spec.numel, model.wl.chunk_symbols, cb, buf[pos:pos + nb]))
        pos += (nb + 15) // 16 * 16
    descs = E.desc_array(descs)
    for _ in range(3):
        E.entro_decode_symbols_batched(descs, packed)
    torch.cuda.synchronize()
    E.entro_profile_begin(steps)
    for _ in range(steps):
        E.entro_decode_symbols_batched(descs, packed)
    torch.cuda.synchronize()
    ms = float(np.mean(E.entro_profile_read(steps)))
    E.entro_profile_begin(0)
    assert E.entro_last_device_status() == E.OK
    bytes_moved = model.stream_bytes + model.index_bytes + model.table_bytes + sum(nbytes)
    return {"kernel_ms": ms, "GBs": bytes_moved / (ms * 1e-3) / 1e9, "weights_per_s": model.n / (ms * 1e-3),
            "output": "two 4-bit symbols per byte" if packed else "one symbol per byte"}


def time_e2e(E, model, steps, warmup):
    """Through the host-buffer entry point: H2D of stream + index, decode, D2H of the fp16 result."""
    descs = model.descs
    n_t = len(descs)
    h_keep, io = [], (E.HostIO * n_t)()
    h2d = d2h = 0
    for i, enc in enumerate(model.keep):
        hs = enc.stream.cpu().pin_memory()
        hi = enc.index.cpu().pin_memory()
        ho = torch.empty(model.out_slices[i].numel(), dtype=torch.float16).pin_memory()
        h_keep += [hs, hi, ho]
        io[i] = E.HostIO(hs.data_ptr(), hi.data_ptr(), ho.data_ptr())
        h2d += hs.numel() * 4 + hi.numel()
        d2h += ho.numel() * 2
    for _ in range(warmup):
        E.entro_decode_dequant_batched_host(descs, io)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(steps):
        E.entro_decode_dequant_batched_host(descs, io)
    ev1.record()
    torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / steps
    # spot check: the host result equals the device result of the device-resident run
    k = min(3, n_t - 1)
    assert torch.equal(h_keep[3 * k + 2], model.out_slices[k].cpu())
    # the same with the result left on the device (a model load from host memory): only the status comes back
    io_load = (E.HostIO * n_t)()
    for i in range(n_t):
        io_load[i] = E.HostIO(io[i].stream_host, io[i].index_host, None)
    E.entro_decode_dequant_batched_host(descs, io_load)
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(steps):
        E.entro_decode_dequant_batched_host(descs, io_load)
        assert E.entro_last_device_status() == E.OK
    ev1.record()
    torch.cuda.synchronize()
    return ms, h2d, d2h, ev0.elapsed_time(ev1) / steps


def measure_gemv(E, max_layers, reps=5, chunk_symbols=0):
    """Config 5: mistral-7B-shaped 4-bit layer stack, batch-1 fp16 GEMV per projection.  Fused
    (decode + dequant + GEMV, one call per layer) against unfused (decode the layer to fp16,
    then seven plain fp16 GEMVs)."""
    wl = workloads.mistral_layer_stack(max_layers=max_layers)
    if chunk_symbols:
        wl = dataclasses.replace(wl, chunk_symbols=chunk_symbols)
    layers = {}
    for spec in wl.tensors:
        layers.setdefault(spec.name.split(".")[1], []).append(spec)
    keep, per_layer, comp_bytes, n_weights = [], [], 0, 0
    biggest = max(sum(t.numel for t in specs) for specs in layers.values())
    scratch = torch.empty(biggest, dtype=torch.float16, device="cuda")
    for name, specs in layers.items():
        descs_f, descs_u, xs, ys, shapes, views = [], [], [], [], [], []
        pos = 0
        for k, spec in enumerate(specs):
            w = workloads.make_tensor(spec, "cuda").view(-1)
            q, qp = E.entro_quantize_tensor(w, wl.bits)
            counts = E.entro_histogram(q, wl.bits)
            cb = E.entro_build_codebook(counts.tolist())
            enc = E.entro_encode(q, cb, wl.chunk_symbols, stream_words=E.entro_stream_words(counts.tolist(), cb))
            del w, q
            keep.append(enc)
            out = scratch[pos:pos + spec.numel]
            pos += spec.numel
            descs_f.append(E.make_desc_no_out(enc.stream, enc.index, spec.numel, wl.chunk_symbols, cb, qp.scale,
                                              qp.zero_point))
            descs_u.append(E.make_desc(enc.stream, enc.index, spec.numel, wl.chunk_symbols, cb, qp.scale,
                                       qp.zero_point, out))
            xs.append(workloads.make_vector(spec.cols, 1000 + k).cuda())
            ys.append(torch.empty(spec.rows, dtype=torch.float16, device="cuda"))
            shapes.append((spec.rows, spec.cols))
            views.append(out.view(spec.rows, spec.cols))
            comp_bytes += (enc.total_bits + 7) // 8 + enc.index.numel() + 2 * (spec.rows + spec.cols)
            n_weights += spec.numel
        per_layer.append((E.desc_array(descs_f), E.desc_array(descs_u), xs, ys, shapes, views,
                          E.make_gemv_io(xs, ys, shapes)))

    def fused():
        for df, du, xs, ys, shapes, views, io in per_layer:
            E.entro_decode_dequant_gemv(df, io=io)

    def unfused():
        for df, du, xs, ys, shapes, views, io in per_layer:
            E.entro_decode_dequant_batched(du)
            for v, x, y in zip(views, xs, ys):
                E.entro_gemv_fp16(v, x, y)

    def timed(fn):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(reps):
            fn()
        ev1.record()
        torch.cuda.synchronize()
        assert E.entro_last_device_status() == E.OK
        return ev0.elapsed_time(ev1) / reps

    plans = [E.entro_gemv_prepare(df, io=io)[0] for df, du, xs, ys, shapes, views, io in per_layer]

    def prepared():
        for plan in plans:
            E.entro_gemv_run(plan)

    out = {"fused": timed(fused), "unfused": timed(unfused), "prepared": timed(prepared)}
    for plan in plans:
        E.entro_gemv_release(plan)
    nl = len(per_layer)

    # Small batches: the same layers with 2, 4, 8 tokens per step.  x of a whole batch must fit the
    # shared-memory staging (batch * cols <= 32768), so the 14336-column projection goes in groups
    # of two tokens: one launch for the six 4096-column projections, one for the groups.
    batches = {}
    for B in (2, 4, 8):
        calls, gemms = [], []
        for df, du, xs, ys, shapes, views, io in per_layer:
            narrow = [k for k, (r, c) in enumerate(shapes) if c * B <= 32768]
            wide = [k for k in range(len(shapes)) if k not in narrow]
            xb = {k: torch.stack([workloads.make_vector(shapes[k][1], 2000 + 31 * k + b) for b in range(B)]).cuda()
                  for k in range(len(shapes))}
            yb = {k: torch.empty(B, shapes[k][0], dtype=torch.float16, device="cuda") for k in range(len(shapes))}
            d1 = E.desc_array([df[k] for k in narrow])
            io1 = E.make_gemv_io([xb[k] for k in narrow], [yb[k] for k in narrow], [shapes[k] for k in narrow])
            calls.append((d1, io1))
            if wide:
                dl, xl, yl, sl = [], [], [], []
                for k in wide:
                    per = max(1, 32768 // shapes[k][1])
                    for b0 in range(0, B, per):
                        dl.append(df[k])
                        xl.append(xb[k][b0:b0 + per])
                        yl.append(yb[k][b0:b0 + per])
                        sl.append(shapes[k])
                calls.append((E.desc_array(dl), E.make_gemv_io(xl, yl, sl)))
            gemms.append((du, [(views[k], xb[k], yb[k]) for k in range(len(shapes))]))

        def fused_b():
            for d, io in calls:
                E.entro_decode_dequant_gemv(d, io=io)

        plans_b = [E.entro_gemv_prepare(d, io=io)[0] for d, io in calls]

        def prepared_b():
            for plan in plans_b:
                E.entro_gemv_run(plan)

        def unfused_b():
            for du, mm in gemms:
                E.entro_decode_dequant_batched(du)
                for w, x, y in mm:
                    torch.matmul(x, w.t(), out=y)

        f, u, pr = timed(fused_b), timed(unfused_b), timed(prepared_b)
        for plan in plans_b:
            E.entro_gemv_release(plan)
        batches[str(B)] = {"fused_ms_per_layer": f / nl, "unfused_ms_per_layer": u / nl,
                           "prepared_ms_per_layer": pr / nl,
                           "prepared_token_weights_per_s": B * n_weights / (pr * 1e-3)}
        del calls, gemms, plans_b
    return {"workload": wl.name, "layers": nl, "weights": n_weights, "chunk_symbols": wl.chunk_symbols,
            "fused_ms_per_layer": out["fused"] / nl, "unfused_ms_per_layer": out["unfused"] / nl,
            "prepared_ms_per_layer": out["prepared"] / nl,
            "speedup_fused_vs_unfused": out["unfused"] / out["fused"],
            "speedup_prepared_vs_unfused": out["unfused"] / out["prepared"],
            "weights_per_s": n_weights / (out["prepared"] * 1e-3),
            "effective_GBs_compressed_in_plus_xy": comp_bytes / (out["prepared"] * 1e-3) / 1e9,
            "fp16_equivalent_GBs": 2.0 * n_weights / (out["prepared"] * 1e-3) / 1e9,
            "batches": batches,
            "note": "fused: entro_decode_dequant_gemv, one call per layer over its 7 projections (descriptor upload, "
                    "table build and decode launch every call); prepared: entro_gemv_prepare once per layer, then "
                    "entro_gemv_run = one launch per layer and token step (the token-generation form; weights_per_s "
                    "and the GB/s figures are the prepared form's); unfused: decode to fp16 then 7 fp16 GEMVs.  The "
                    "fused pass is bound by decode issue rate, not by HBM (0.14 B/weight read).  batches: 2, 4, 8 "
                    "tokens per step (two launches per layer) against decode + 7 library GEMMs"}


def measure_other(E, name, steps, peak):
    """One of the other configurations, briefly: its own model build, a few warm-up passes, `steps`
    timed passes (CUDA events around the whole step, and the library's events around the decode
    kernel alone).  Outside the headline's timed region."""
    wl = pick_workload(name, None)
    model = DeviceModel(wl, E, E.DEFAULT_DECODE_CONFIG[0])
    for _ in range(3):
        E.entro_decode_dequant_batched(model.descs)
    torch.cuda.synchronize()
    E.entro_profile_begin(steps)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        E.entro_decode_dequant_batched(model.descs)
    ev1.record()
    torch.cuda.synchronize()
    step_ms = ev0.elapsed_time(ev1) / steps
    kernel_ms = E.entro_profile_read(steps)
    E.entro_profile_begin(0)
    assert E.entro_last_device_status() == E.OK
    k_ms = float(np.mean(kernel_ms))
    achieved = model.algorithmic_bytes / (k_ms * 1e-3) / 1e9
    in_l2 = model.algorithmic_bytes < 100e6
    out = {"workload": wl.name + " full-model decode", "bits": wl.bits, "chunk_symbols": wl.chunk_symbols,
           "tensors": len(wl.tensors), "weights": model.n, "bits_per_weight": model.bits_per_weight,
           "max_code_len": model.max_len, "steps": steps, "ms_per_step": step_ms,
           "value": model.algorithmic_bytes / (step_ms * 1e-3) / 1e9, "unit": "GB/s",
           "weights_per_s": model.n / (step_ms * 1e-3), "bytes_per_step": model.algorithmic_bytes,
           "roofline": {"bound": "hbm", "kernel": "decode_kernel", "achieved": achieved, "peak": peak[0], "unit": "GB/s",
                        "frac": achieved / peak[0], "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS, "kernel_ms": k_ms,
                        "kernel_ms_min": float(np.min(kernel_ms))}}
    if in_l2:
        # the timed calls above repeat one call, which finds descriptors and tables in place (one launch);
        # two alternating calls (same tensor, two output buffers) rebuild them every time
        import ctypes as C
        out2 = torch.empty_like(model.out)
        alt = (E.TensorDesc * len(model.descs))()
        for i, d in enumerate(model.descs):
            C.memmove(C.byref(alt[i]), C.byref(d), C.sizeof(E.TensorDesc))
            alt[i].out_fp16_dev = out2.data_ptr() + (d.out_fp16_dev - model.out.data_ptr())
        for _ in range(3):
            E.entro_decode_dequant_batched(model.descs)
            E.entro_decode_dequant_batched(alt)
        torch.cuda.synchronize()
        ev0.record()
        for _ in range(steps):
            E.entro_decode_dequant_batched(model.descs)
            E.entro_decode_dequant_batched(alt)
        ev1.record()
        torch.cuda.synchronize()
        assert E.entro_last_device_status() == E.OK and torch.equal(out2, model.out)
        out["us_per_call"] = 1e3 * step_ms
        out["us_per_call_tables_rebuilt"] = 1e3 * ev0.elapsed_time(ev1) / (2 * steps)
        out["note"] = ("latency-bound: the whole tensor (%.1f MB of traffic) stays in L2 and a call is a handful of "
                       "microseconds of launches, so the roofline fraction is not a roofline point.  us_per_call: the "
                       "same call repeated (descriptors and tables found in place, one launch); "
                       "us_per_call_tables_rebuilt: descriptor upload + table build + decode every call"
                       % (model.algorithmic_bytes / 1e6))
    del model
    torch.cuda.empty_cache()
    return out


# ----------------------------------------------------------------------------- CPU oracle legs

def oracle_sample(wl, max_symbols):
    """First matrices of the workload up to max_symbols, compressed BY THE ORACLE on the host."""
    import oracle
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    items, total = [], 0
    for spec in wl.matrices():
        if not spec.name.startswith("layers."):
            continue
        if items and total + spec.numel > max_symbols:
            break
        w = workloads.make_tensor(spec, dev).view(-1).cpu().numpy()
        c = oracle.compress(w, wl.bits, wl.chunk_symbols)
        items.append((spec, c))
        total += spec.numel
    nbytes = 0
    for spec, c in items:
        nch = oracle.num_chunks(spec.numel, wl.chunk_symbols)
        nbytes += (c.enc.total_bits + 7) // 8 + 8 * (nch + 1) + 64 * nch + 2 * spec.numel
    return items, total, nbytes


def oracle_pass(wl, items, threads):
    import oracle
    t0 = time.perf_counter()
    for spec, c in items:
        oracle.decode_dequant(c.enc.stream, c.enc.offsets, spec.numel, wl.chunk_symbols, c.lengths,
                              c.qp.scale, c.qp.zero_point, want_q=False, threads=threads)
    return time.perf_counter() - t0


def cpu_baseline(wl, budget_cpu_s=12.0):
    threads = os.cpu_count() or 1
    items, nsym, nbytes = oracle_sample(wl, 120_000_000)
    oracle_pass(wl, items[:1], threads)        # touch code and pages
    passes, wall = 0, 0.0
    while wall * threads < budget_cpu_s and wall < 60.0:
        wall += oracle_pass(wl, items, threads)
        passes += 1
    names = ", ".join(s.name for s, _ in items)
    # the paper's own thread count (4, Section 4) and one thread, on the first tensor of the sample, one pass each
    spec0, c0 = items[0]
    bytes0 = nbytes * spec0.numel / nsym
    fewer = {}
    for t in (4, 1):
        w = oracle_pass(wl, items[:1], t)
        fewer[str(t)] = {"value": bytes0 / w / 1e9, "weights_per_s": spec0.numel / w, "seconds": w}
    return {"value": nbytes * passes / wall / 1e9, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "weights_per_s": nsym * passes / wall,
            "sample": f"{names} of {wl.name} ({nsym} weights), bit-serial decode + dequant, chunks dealt "
                      f"round-robin to {threads} threads, {passes} passes in {wall:.2f} s",
            "fewer_threads": fewer, "fewer_threads_sample": f"{spec0.name} ({spec0.numel} weights), one pass"}


def run_reference(args, rank, world):
    """The reference arm: the CPU oracle as it stands, on the host cores, rank 0 only."""
    if rank != 0:
        return
    wl = pick_workload(args.workload, args.max_layers)
    threads = os.cpu_count() or 1
    items, nsym, nbytes = oracle_sample(wl, 45_000_000)
    for _ in range(args.warmup):
        oracle_pass(wl, items, threads)
    t = 0.0
    for _ in range(args.steps):
        t += oracle_pass(wl, items, threads)
    value = nbytes * args.steps / t / 1e9
    names = ", ".join(s.name for s, _ in items)
    sample = (f"each step: {names} of {wl.name} ({nsym} weights), bit-serial decode + dequant on "
              f"{threads} host threads")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
        "config": {"workload": wl.name + " full-model decode (bounded sample per step)", "bits": wl.bits,
                   "chunk_symbols": wl.chunk_symbols},
        "weights_per_s": nsym * args.steps / t,
        "cpu_baseline": {"value": value, "unit": "GB/s", "kind": "oracle", "cores": threads, "sample": sample},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


# ----------------------------------------------------------------------------- main

def measure(E, wl, args, world, local_rank, rank, peak, with_e2e, with_cpu):
    model = DeviceModel(wl, E, args.lut_bits, max_code_len=args.max_code_len)
    ms, launches, kernel_ms, clocks = time_steps(E, model, args.steps, args.warmup, world,
                                                 physical_gpu_index(local_rank))
    ms_step = ms / args.steps
    value = world * model.algorithmic_bytes / (ms_step * 1e-3) / 1e9
    k_ms = float(np.mean(kernel_ms)) if kernel_ms else ms_step
    achieved = model.algorithmic_bytes / (k_ms * 1e-3) / 1e9
    res = {
        "value": value, "ms_per_step": ms_step, "weights_per_s": world * model.n / (ms_step * 1e-3),
        "bytes_per_step": model.algorithmic_bytes, "bits_per_weight": model.bits_per_weight,
        "max_code_len": model.max_len, "gpu_launches": int(launches), "clocks": clocks,
        "roofline": {"bound": "hbm", "kernel": "decode_kernel", "achieved": achieved, "peak": peak[0],
                     "unit": "GB/s", "frac": achieved / peak[0], "peak_source": peak[1],
                     "frac_of_nominal_8000": achieved / NOMINAL_HBM_GBS, "kernel_ms": k_ms,
                     "kernel_ms_min": float(np.min(kernel_ms)) if kernel_ms else None,
                     "kernel_ms_median": float(np.median(kernel_ms)) if kernel_ms else None,
                     "traffic": (NCU_DRAM_BYTES_PER_WEIGHT.get(wl.bits) * model.n
                                 if NCU_DRAM_BYTES_PER_WEIGHT.get(wl.bits) else None),
                     "traffic_note": "bytes per launch: ncu DRAM read+write on the 1-layer case, scaled by weights"},
        "compress": {"seconds": model.compress_s, "weights_per_s": model.n / model.compress_s, **model.compress_stages,
                     "what": "entro_quantize_histogram_batched + codebooks (host) + entro_encode_batched over the whole "
                             "resident fp16 model, wall clock, one synchronise per stage; outside the timed steps"},
        "model": model,
    }
    if with_e2e and rank == 0 or (with_e2e and world > 1):
        e_ms, h2d, d2h, load_ms = time_e2e(E, model, max(1, min(args.e2e_steps, args.steps)), 1)
        res["e2e"] = {"value": world * model.algorithmic_bytes / (e_ms * 1e-3) / 1e9, "unit": "GB/s",
                      "ms_per_step": e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                      "result_left_on_device": {"value": world * model.algorithmic_bytes / (load_ms * 1e-3) / 1e9,
                                                "unit": "GB/s", "ms_per_step": load_ms, "h2d_bytes_per_step": h2d,
                                                "d2h_bytes_per_step": 4,
                                                "what": "same call without host output buffers (a model load from "
                                                        "pinned host memory); only the status word is read back"}}
    if rank == 0 and world == 1:
        res["symbols_out"] = time_symbols(E, model)
    if with_cpu and rank == 0 and world == 1:
        res["cpu_baseline"] = cpu_baseline(wl)
    return res


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="own", choices=["own", "reference"])
    ap.add_argument("--workload", default="mistral8",
                    choices=["mistral8", "mistral4", "smollm8", "phi3_4", "single", "mistral8-gauss", "mistral4-gauss",
                             "mistral8-paperbits", "mistral4-paperbits"])
    ap.add_argument("--also", default="mistral4", help="second workload reported under 'also' ('' = none)")
    ap.add_argument("--max-layers", type=int, default=None, help="truncate the model (for profiling runs)")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--no-gemv", action="store_true", help="skip the fused decode+GEMV section (config 5)")
    ap.add_argument("--others", default="smollm8,phi3_4,single,mistral8-paperbits,mistral4-paperbits",
                    help="further workloads, each timed briefly and listed under 'others' ('' = none)")
    ap.add_argument("--others-steps", type=int, default=10)
    ap.add_argument("--max-code-len", type=int, default=0,
                    help="use length-limited codes (not the paper's optimal code); 0 = unrestricted Huffman")
    ap.add_argument("--chunk-symbols", type=int, default=0,
                    help="code the main workload with this chunk size instead of its own (a multiple of 256)")
    ap.add_argument("--gemv-chunk-symbols", type=int, default=0, help="chunk size of the fused-GEMV section's streams")
    ap.add_argument("--lut-bits", type=int, default=0)
    ap.add_argument("--warps", type=int, default=0)
    ap.add_argument("--ctas", type=int, default=0)
    ap.add_argument("--item", type=int, default=0)
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import paper_2505_02380_b200 as E   # fails loudly if the CUDA library is not built
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    E.lib()
    if args.lut_bits or args.warps or args.ctas or args.item:
        E.entro_set_decode_config(args.lut_bits, args.warps, args.ctas, args.item)
    if not args.lut_bits:
        args.lut_bits = E.DEFAULT_DECODE_CONFIG[0]
    peak = measured_peak()

    wl = pick_workload(args.workload, args.max_layers)
    if args.chunk_symbols:
        wl = dataclasses.replace(wl, chunk_symbols=args.chunk_symbols)
    main_res = measure(E, wl, args, world, local_rank, rank, peak, not args.no_e2e, not args.no_cpu)
    main_res.pop("model")
    also = None
    if args.also and args.also != args.workload:
        torch.cuda.empty_cache()
        wl2 = pick_workload(args.also, args.max_layers)
        r2 = measure(E, wl2, args, world, local_rank, rank, peak, False, False)
        r2.pop("model")
        also = {"workload": wl2.name + " full-model decode", "bits": wl2.bits, "chunk_symbols": wl2.chunk_symbols,
                **{k: r2[k] for k in ("value", "ms_per_step", "weights_per_s", "bytes_per_step", "bits_per_weight",
                                       "max_code_len", "roofline", "clocks", "symbols_out") if k in r2}}

    gemv = None
    if not args.no_gemv and rank == 0 and world == 1:
        torch.cuda.empty_cache()
        gemv = measure_gemv(E, args.max_layers, chunk_symbols=args.gemv_chunk_symbols)

    others = []
    if args.others and rank == 0 and world == 1:
        for name in args.others.split(","):
            if name and name not in (args.workload, args.also):
                torch.cuda.empty_cache()
                others.append(measure_other(E, name, args.others_steps, peak))

    if rank == 0:
        line = {
            "metric": METRIC, "value": main_res["value"], "unit": "GB/s", "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": main_res["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "u32", "data": "synthetic",
            "config": {"workload": wl.name + " full-model decode", "bits": wl.bits,
                       "chunk_symbols": wl.chunk_symbols, "tensors": len(wl.tensors), "weights": wl.numel,
                       "max_layers": args.max_layers, "lut_bits": args.lut_bits, "max_code_len_cap": args.max_code_len,
                       "l2": "inputs and outputs per step (GBs) are far larger than L2; no flush needed",
                       "parallelism": f"replicas x{world}, one full model per GPU, no collective"},
            "weights_per_s": main_res["weights_per_s"], "bytes_per_step": main_res["bytes_per_step"],
            "bits_per_weight": main_res["bits_per_weight"], "max_code_len": main_res["max_code_len"],
            "pct_of_nominal_8000_GBs": 100.0 * main_res["value"] / world / NOMINAL_HBM_GBS,
            "pct_of_measured_copy": 100.0 * main_res["value"] / world / peak[0],
            "roofline": main_res["roofline"], "clocks": main_res["clocks"],
            "gpu_launches": main_res["gpu_launches"],
        }
        if "e2e" in main_res:
            line["e2e"] = main_res["e2e"]
        if "cpu_baseline" in main_res:
            line["cpu_baseline"] = main_res["cpu_baseline"]
        if "symbols_out" in main_res:
            line["symbols_out"] = main_res["symbols_out"]
        line["compress"] = main_res["compress"]
        if also:
            line["also"] = also
        if gemv:
            line["gemv"] = gemv
        if others:
            line["others"] = others
        line["paper_context"] = ("paper: 6.66 s (uint8) / 1.66 s (uint4) to decode phi3-mini-4k on a Jetson P3450, "
                                 "4 CPU threads, integer output (Table 3) -- other hardware, context only")
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

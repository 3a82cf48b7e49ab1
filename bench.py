#!/usr/bin/env python
"""Benchmark of the activation codec on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

A step is one pass of the whole hot path over one batch of synthetic activations: for every code
width b in {2, 4, 8}, compress every tensor of the workload (forward order), then decompress every
one (reverse order), salient_mode AUTO.  The headline workload is the ResNet-18-shaped set of saved
activations at batch 64 (17 fp32 tensors, 563.5 MiB dense).  `value` is dense GB/s: the dense bytes
that went through compress plus those that came out of decompress, divided by the device time.

Beside the headline the line carries `sweep` (the size sweep of configs[3]: single tensors of 64 MiB, 256 MiB and
1 GiB, fp32 and bf16, compress and decompress timed separately over copies that do not fit the L2 cache),
`schedule` (configs[4] through fh_run_schedule) and `parity_checked` (status words re-read after the timed
region and one tensor's container per code width compared byte for byte with the CPU oracle).

One JSON line goes to stdout (rank 0).  With N > 1 (launched by torchrun) every rank runs the
same workload on its own GPU -- planes and tensors are independent, there is no exchange step --
and the value is the sum of the dense bytes over the slowest rank's time.
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

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_11400_b200 import synth  # noqa: E402

BITS = (2, 4, 8)
# dram__bytes_read.sum + dram__bytes_write.sum per compress call (one kernel), averaged over the 51 compress calls
# of a step of the default workload; see profiles/compress_resnet18_b64_traffic.md.  None: the kernels have
# changed since the counters were taken.
NCU_DRAM_BYTES_PER_COMPRESS_CALL = 35842424
METRIC = "compress+decompress throughput, dense activation bytes"
UNIT = "GB/s"


def workload_specs(name: str):
    if name == "resnet18_b64":
        return synth.config2(64), "configs[1]: ResNet-18-shaped saved activations, batch 64, 224x224 input, fp32, " \
                                  "17 tensors, 563.5 MiB dense; even tensors ReLU(N(0,1)), odd N(0,1)"
    if name == "mobilenetv2_b128":
        return synth.config3(128), "configs[2]: MobileNetV2-shaped expanded activations, batch 128, bf16, Laplace(0,1) " \
                                   "with channel-clustered +-50 outliers"
    if name == "mobilenetv2_b128_iid":
        return synth.config3(128, stress=True), "configs[2]: MobileNetV2-shaped expanded activations, batch 128, bf16, " \
                                                "Laplace(0,1) with 1 % outliers at +-50, independent per element"
    if name == "cifar_schedule":
        return synth.config5(128), "configs[4]: 20 ResNet-18/CIFAR-shaped tensors, batch 128, fp32"
    if name == "config1":
        return synth.config1(), "configs[0]: 32x16x32x32 fp32 ReLU(N(0,1))"
    if name.startswith("sweep_"):          # sweep_<MiB>_<f32|bf16>
        _, mib, dt = name.split("_")
        return synth.config4(int(mib), synth.F32 if dt == "f32" else synth.BF16), \
            f"configs[3]: single {mib} MiB {dt} tensor of 32x32 planes, ReLU(N(0,1))"
    if name.startswith("shape_"):          # shape_<n>x<c>x<h>x<w>_<f32|bf16>_<kind>: one tensor, for profiling
        _, dims, dt, kind = name.split("_", 3)
        shape = tuple(int(v) for v in dims.split("x"))
        return [synth.TensorSpec("shape", shape, synth.F32 if dt == "f32" else synth.BF16, kind, 900)], \
            f"single {dt} tensor {dims}, {kind}"
    raise SystemExit(f"unknown workload {name}")


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def slowest_rank(value: float, world: int, device=None) -> float:
    """The timing rule for N replicas: every rank contributes its own device time, the job's time is the
    slowest rank's.  (One all-reduce(MAX) of a scalar; the data path itself has no collective.)"""
    if world <= 1:
        return float(value)
    import torch
    import torch.distributed as dist
    t = torch.tensor([float(value)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(dense_bytes_per_rank: int, world: int, seconds: float) -> float:
    """Aggregate dense GB/s of N replicas that each pushed `dense_bytes_per_rank` through the codec."""
    return world * dense_bytes_per_rank / seconds / 1e9


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = "clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown," \
        "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown," \
        "clocks_event_reasons.sw_power_cap"

    def __init__(self, index: int):
        self.rows = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([c.strip() for c in line.split(",")])

    def keep_busy(self, step, want: int, limit_s: float):
        """Repeats `step` (untimed) until `want` samples have come in or `limit_s` seconds have passed: the
        timed region of a short run is over before nvidia-smi has answered once, so the same load is kept up
        on both sides of it and the samples are those of that load."""
        if self.proc is None:
            return
        import torch
        t0 = time.perf_counter()
        while len(self.rows) < want and time.perf_counter() - t0 < limit_s:
            step()
            torch.cuda.synchronize()

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except Exception:
                continue
            for n, v in zip(names, r[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------------------
# reference arm: the CPU oracle, as it stands, on a bounded sample of the same workload
# ------------------------------------------------------------------------------------------------

def oracle_sample(specs, frac_planes: float):
    """First planes of every tensor of the workload (planes are coded independently, so a prefix of
    the batch is the same work per byte)."""
    out = []
    for s in specs:
        n, c, h, w = s.shape
        P = n * c
        take = max(1, min(P, int(round(P * frac_planes))))
        sub = synth.TensorSpec(s.name, (1, take, h, w), s.dtype, s.kind, s.seed)
        out.append((sub, synth.make(sub)))
    return out


def time_oracle(sample, threads: int):
    from oracle import fho
    fho.set_threads(threads)
    dense = 0
    t0 = time.perf_counter()
    for b in BITS:
        p = fho.params(bits=b)
        packed = []
        for sub, raw in sample:
            d = fho.desc(sub.shape, sub.dtype)
            st, buf, total = fho.compress(raw, d, p)
            assert st == 0
            packed.append((d, buf))
            dense += raw.nbytes
        for d, buf in reversed(packed):
            st, out = fho.decompress(buf, d)
            assert st == 0
            dense += out.nbytes
    return dense, time.perf_counter() - t0


def cpu_baseline(specs, budget_s: float = 15.0):
    from oracle import fho
    cores = fho.max_threads()
    probe = oracle_sample(specs, 0.01)
    dense, t = time_oracle(probe, cores)
    rate = dense / max(t, 1e-6)
    total_dense = sum(s.dense_bytes for s in specs) * 2 * len(BITS)
    frac = min(1.0, budget_s * rate / total_dense)
    sample = oracle_sample(specs, frac)
    dense, t = time_oracle(sample, cores)
    return {"value": dense / t / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {frac * 100:.2f}% of the planes of every tensor, bits 2/4/8, compress+decompress, "
                      f"{dense / 2 / len(BITS) / 2**20:.1f} MiB dense per pass, {t:.1f} s"}


def run_reference(args, specs, wl_desc):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import fho
    cores = fho.max_threads()
    probe = oracle_sample(specs, 0.01)
    dense, t = time_oracle(probe, cores)
    rate = dense / max(t, 1e-6)
    total_dense = sum(s.dense_bytes for s in specs) * 2 * len(BITS)
    budget = 120.0 / max(1, args.steps + args.warmup)
    frac = min(1.0, budget * rate / total_dense)
    sample = oracle_sample(specs, frac)
    for _ in range(args.warmup):
        time_oracle(sample, cores)
    tot_d, tot_t = 0, 0.0
    for _ in range(args.steps):
        d, t = time_oracle(sample, cores)
        tot_d += d
        tot_t += t
    val = tot_d / tot_t / 1e9
    smp = f"first {frac * 100:.3f}% of the planes of every tensor per step ({tot_d / args.steps / 2**20:.1f} MiB dense " \
          f"through the codec per step)"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": tot_t / args.steps * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl_desc, "bits": list(BITS), "salient_mode": "AUTO", "sample": smp},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": smp},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------------
# our arm
# ------------------------------------------------------------------------------------------------

def size_sweep(api, peak, mibs=(64, 256, 1024), repeats=20):
    """configs[3]: single tensors of 32x32 planes, ReLU(N(0,1)), 2 bits, three-sigma mode; compress and
    decompress timed separately with CUDA events over back-to-back calls on copies that together exceed the L2
    cache.  fraction = (dense + container bytes) / time / measured copy bandwidth."""
    import ctypes as C
    import torch
    L = api.lib()
    sp = int(torch.cuda.current_stream().cuda_stream)
    out = {}
    for dt, dname in ((synth.F32, "f32"), (synth.BF16, "bf16")):
        for mib in mibs:
            spec = synth.config4(mib, dt)[0]
            raw = synth.make(spec)
            base = torch.from_numpy(raw.view(np.int16) if raw.dtype == np.uint16 else raw).cuda()
            d = api.desc(spec.shape, spec.dtype)
            p = api.default_params(bits=2)
            cap = api.compressed_bytes(d, p, 1)
            ncopy = max(2, -(-(400 << 20) // spec.dense_bytes))
            copies = [base] + [base.clone() for _ in range(ncopy - 1)]
            packs = [torch.empty(cap, dtype=torch.uint8, device="cuda") for _ in range(ncopy)]
            rest = torch.empty_like(base)
            out2 = torch.zeros(2, dtype=torch.int64, device="cuda")
            st = torch.zeros(1, dtype=torch.int64, device="cuda")
            cargs = [(C.byref(d), C.byref(p), c.data_ptr(), k.data_ptr(), cap, out2.data_ptr(), sp) for c, k in zip(copies, packs)]
            dargs = [(k.data_ptr(), cap, C.byref(d), rest.data_ptr(), st.data_ptr(), sp) for k in packs]
            reps = -(-repeats // ncopy)
            res = {}
            for name, arglist, fn in (("compress", cargs, L.fh_compress), ("decompress", dargs, L.fh_decompress)):
                for a in arglist * 2:       # warm-up
                    assert fn(*a) == 0
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    for a in arglist:
                        assert fn(*a) == 0
                e1.record()
                torch.cuda.synchronize()
                assert out2[1].item() == 0 and st.item() == 0
                res[name] = e0.elapsed_time(e1) * 1e-3 / (reps * ncopy)
            total = int(out2[0].item())
            out[f"{mib}MiB_{dname}"] = {
                "dense_bytes": spec.dense_bytes, "packed_bytes": total, "calls_timed": reps * ncopy,
                "compress_gbs": spec.dense_bytes / res["compress"] / 1e9,
                "decompress_gbs": spec.dense_bytes / res["decompress"] / 1e9,
                "compress_frac": (spec.dense_bytes + total) / res["compress"] / 1e9 / peak,
                "decompress_frac": (spec.dense_bytes + total) / res["decompress"] / 1e9 / peak}
            del copies, packs, rest, base
            torch.cuda.empty_cache()
    return out


def schedule_leg(api, mode, repeats=20):
    """configs[4]: the 20 CIFAR-ResNet-shaped tensors at batch 128, every other one compressed, through
    fh_run_schedule (forward-order compress, reverse-order decompress, one stream)."""
    import torch
    specs = synth.config5(128)
    p = api.default_params(bits=2, salient_mode=mode)
    items, need = [], 0
    for i, s in enumerate(specs):
        t = torch.from_numpy(synth.make(s)).cuda()
        d = api.desc(s.shape, s.dtype, tensor_id=i)
        items.append(api.SchedItem(d, api.FH_COMPRESS if s.compress else api.FH_KEEP, t, torch.empty_like(t)))
        if s.compress:
            need += (api.compressed_bytes(d, p, 1) + 255) & ~255
    arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    for _ in range(3):
        rep = api.fh_run_schedule(items, p, arena)
        assert rep.status == api.FH_OK, rep.status
    fwd = bwd = 0.0
    for _ in range(repeats):
        rep = api.fh_run_schedule(items, p, arena)
        assert rep.status == api.FH_OK, rep.status
        fwd += rep.ms_forward
        bwd += rep.ms_backward
    dense = int(rep.total_dense_bytes)
    return {"tensors": len(specs), "compressed_tensors": sum(1 for s in specs if s.compress), "repeats": repeats,
            "ms_forward": fwd / repeats, "ms_backward": bwd / repeats, "total_dense_bytes": dense,
            "total_packed_bytes": int(rep.total_packed_bytes), "peak_packed_bytes": int(rep.peak_packed_bytes),
            "compress_gbs": dense / (fwd / repeats) / 1e6, "decompress_gbs": dense / (bwd / repeats) / 1e6}


def run_ours(args, specs, wl_desc):
    import torch
    import torch.distributed as dist
    from paper_2510_11400_b200 import api, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    api.lib()

    # the oracle is timed first (rank 0, N = 1 only), before the GPU is busy
    cpu = cpu_baseline(specs) if (rank == 0 and world == 1 and not args.no_cpu) else None

    dev = torch.device("cuda", local)
    mode = {"auto": api.FH_SALIENT_AUTO, "off": api.FH_SALIENT_OFF, "all": api.FH_SALIENT_ALL,
            "channel": api.FH_SALIENT_CHANNEL, "tensor": api.FH_SALIENT_TENSOR}[args.mode]
    params = {b: api.default_params(bits=b, salient_mode=mode, rounding=args.rounding, seed=2510_11400) for b in BITS}
    tensors = []
    for i, s in enumerate(specs):
        raw = synth.make(s)
        t = torch.from_numpy(raw.view(np.int16) if raw.dtype == np.uint16 else raw).to(dev)
        d = api.desc(s.shape, s.dtype, tensor_id=i)
        cap = api.compressed_bytes(d, params[8], 1)
        tensors.append(dict(spec=s, desc=d, dense=t, packed=torch.empty(cap, dtype=torch.uint8, device=dev),
                            restored=torch.empty_like(t), cap=cap,
                            out2={b: torch.zeros(2, dtype=torch.int64, device=dev) for b in BITS},
                            st={b: torch.zeros(1, dtype=torch.int64, device=dev) for b in BITS}))
    dense_bytes = sum(s.dense_bytes for s in specs)
    n_tensors = len(tensors)
    stream = torch.cuda.current_stream()

    # argument tuples are marshalled once: the timed loop only makes the C calls
    import ctypes as C
    L = api.lib()
    sp = int(stream.cuda_stream)
    cargs = {b: [(C.byref(t["desc"]), C.byref(params[b]), t["dense"].data_ptr(), t["packed"].data_ptr(), t["cap"],
                  t["out2"][b].data_ptr(), sp) for t in tensors] for b in BITS}
    dargs = {b: [(t["packed"].data_ptr(), t["cap"], C.byref(t["desc"]), t["restored"].data_ptr(), t["st"][b].data_ptr(), sp)
                 for t in reversed(tensors)] for b in BITS}

    def step(ev=None):
        for b in BITS:
            if ev is not None:
                ev[b][0].record(stream)
            for a in cargs[b]:
                rc = L.fh_compress(*a)
                assert rc == 0, rc
            if ev is not None:
                ev[b][1].record(stream)
            for a in dargs[b]:
                rc = L.fh_decompress(*a)
                assert rc == 0, rc
            if ev is not None:
                ev[b][2].record(stream)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    packed_bytes = {}
    for b in BITS:
        tot = 0
        for t in tensors:
            total, st = t["out2"][b].tolist()
            assert st == 0, f"device status {st}"
            assert t["st"][b].item() == 0
            tot += total
        packed_bytes[b] = tot

    evs = [{b: [torch.cuda.Event(enable_timing=True) for _ in range(3)] for b in BITS} for _ in range(args.steps)]
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    sampler.start()
    if not args.no_clock_window:
        sampler.keep_busy(step, 2, 3.0)  # (untimed) the load is running when the first samples are taken
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = api.kernel_launches()
    e0.record(stream)
    for k in range(args.steps):
        step(evs[k])
    e1.record(stream)
    torch.cuda.synchronize()
    launches = api.kernel_launches() - launches0
    if world > 1:
        dist.barrier()
    if not args.no_clock_window:
        sampler.keep_busy(step, len(sampler.rows) + 4, 1.5)  # (untimed) ... and still running for the last ones
    clocks = sampler.stop()
    if not args.no_clock_window:
        clocks["window"] = "the same step repeated back to back, untimed, before and after the timed steps"
    ms = e0.elapsed_time(e1)
    ms = slowest_rank(ms, world, dev)
    t_comp = {b: sum(e[b][0].elapsed_time(e[b][1]) for e in evs) for b in BITS}
    t_dec = {b: sum(e[b][1].elapsed_time(e[b][2]) for e in evs) for b in BITS}

    # ---- after the timed region: every status word again, and one tensor per code width against the oracle
    for b in BITS:
        for t in tensors:
            total, st = t["out2"][b].tolist()
            assert st == 0 and t["st"][b].item() == 0, f"device status after the timed region: {st}, {t['st'][b].item()}"
    parity_checked = False
    if rank == 0 and not args.no_cpu:
        from oracle import fho
        fho.set_threads(fho.max_threads())
        k = min(len(tensors) - 1, 10)         # a tensor of small planes when the workload has one (mixed plane classes)
        t = tensors[k]
        raw = synth.make(t["spec"])
        for b in BITS:
            assert L.fh_compress(*cargs[b][k]) == 0
            torch.cuda.synchronize()
            total = int(t["out2"][b][0])
            st_o, buf_o, total_o = fho.compress(raw, fho.desc(t["spec"].shape, t["spec"].dtype, tensor_id=k),
                                                fho.params(bits=b, salient_mode=mode, rounding=args.rounding, seed=2510_11400))
            assert st_o == 0 and total == total_o, (total, total_o)
            assert np.array_equal(t["packed"][:total].cpu().numpy(), buf_o), "container differs from the oracle's"
            assert L.fh_decompress(t["packed"].data_ptr(), t["cap"], C.byref(t["desc"]), t["restored"].data_ptr(),
                                   t["st"][b].data_ptr(), sp) == 0
            torch.cuda.synchronize()
            got = t["restored"].cpu().numpy()
            _, out_o = fho.decompress(buf_o, fho.desc(t["spec"].shape, t["spec"].dtype))
            assert np.array_equal(got.view(np.uint16) if t["spec"].dtype == synth.BF16 else got.view(np.uint32),
                                  out_o if t["spec"].dtype == synth.BF16 else out_o.view(np.uint32)), "restored values differ"
        parity_checked = True

    # ---- end to end through the host-buffer entry points (pinned host memory on both sides)
    e2e = None
    if not args.no_e2e:
        work = torch.empty(max(api.host_work_bytes(t["desc"], params[8]) for t in tensors), dtype=torch.uint8, device=dev)
        hosts = []
        for t in tensors:
            hosts.append(dict(src=t["dense"].cpu().pin_memory(), pack=torch.empty(t["cap"], dtype=torch.uint8).pin_memory(),
                              out=torch.empty_like(t["dense"], device="cpu").pin_memory()))
        def e2e_step():
            h2d = d2h = 0
            for b in BITS:
                sizes = []
                for t, h in zip(tensors, hosts):
                    st, total = api.fh_compress_host(t["desc"], params[b], h["src"], h["pack"], work)
                    assert st == 0, st
                    sizes.append(total)
                    h2d += t["spec"].dense_bytes
                    d2h += total + 16
                for t, h, total in reversed(list(zip(tensors, hosts, sizes))):
                    st = api.fh_decompress_host(h["pack"], total, t["desc"], h["out"], work)
                    assert st == 0, st
                    h2d += total
                    d2h += t["spec"].dense_bytes + 8
            return h2d, d2h
        e2e_step()
        ksteps = max(1, min(args.steps, 3))
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(ksteps):
            h2d, d2h = e2e_step()
        torch.cuda.synchronize()
        dt = time.perf_counter() - t0
        dt = slowest_rank(dt, world, dev)
        e2e = {"value": whole_job_value(ksteps * dense_bytes * 2 * len(BITS), world, dt), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": ksteps}

    sweep = sched = None
    if rank == 0 and world == 1 and args.workload == "resnet18_b64" and not args.no_sweep:
        del tensors, cargs, dargs
        torch.cuda.empty_cache()
        sweep = size_sweep(api, peaks()[0])
        sched = schedule_leg(api, mode)

    if rank == 0:
        peak, peak_kind = peaks()
        n_comp = args.steps * len(BITS) * n_tensors
        alg_comp = args.steps * sum(dense_bytes + packed_bytes[b] for b in BITS)
        comp_s = sum(t_comp.values()) / 1e3
        achieved = alg_comp / comp_s / 1e9
        # DRAM bytes per compress call from the ncu capture summarised under profiles/ (null for any other
        # workload or mode than the one captured)
        traffic = NCU_DRAM_BYTES_PER_COMPRESS_CALL if (args.workload == "resnet18_b64" and args.mode == "auto") else None
        value = whole_job_value(args.steps * dense_bytes * 2 * len(BITS), world, ms / 1e3)
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32" if specs[0].dtype == synth.F32 else "bf16", "data": "synthetic",
            "config": {"workload": wl_desc + ("; every tensor compressed" if args.workload == "cifar_schedule" else ""),
                       "bits": list(BITS), "salient_mode": args.mode.upper(),
                       "rounding": "nearest-even" if args.rounding == 0 else "random (Philox-4x32-10)",
                       "tensors": n_tensors, "dense_bytes_per_pass": dense_bytes,
                       "packed_bytes": {str(b): packed_bytes[b] for b in BITS},
                       "l2": "inputs larger than L2: every pass streams the whole dense set",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "compress_gbs": {str(b): args.steps * dense_bytes / t_comp[b] / 1e6 for b in BITS},
            "decompress_gbs": {str(b): args.steps * dense_bytes / t_dec[b] / 1e6 for b in BITS},
            "roofline": {"bound": "hbm",
                         "kernel": "compress call = one kernel (compress_warp / compress_cta_regs / compress_cta / compress_generic by plane "
                                   "size); averaged over every compress call of the timed region",
                         "achieved": achieved, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak, "traffic": traffic,
                         "launches": n_comp, "avg_launch_us": comp_s / n_comp * 1e6,
                         "algorithmic_bytes_per_launch": alg_comp / n_comp,
                         "frac_of_nominal_8000": achieved / 8000.0,
                         "decompress_achieved": args.steps * sum(dense_bytes + packed_bytes[b] for b in BITS)
                         / (sum(t_dec.values()) / 1e3) / 1e9},
            "clocks": clocks, "gpu_launches": int(launches), "parity_checked": parity_checked,
        }
        if sweep is not None:
            line["sweep"] = sweep
        if sched is not None:
            line["schedule"] = sched
        if e2e is not None:
            line["e2e"] = e2e
        if cpu is not None:
            line["cpu_baseline"] = cpu
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    api.shutdown()


def run_schedule(args, specs, wl_desc):
    """One training step's worth of codec work through fh_run_schedule: the tensors marked `compress` are
    compressed in forward order into one arena and restored in reverse order, on one stream.  A step is one
    call; the library times the two phases with CUDA events and reports the arena's high-water mark."""
    import torch
    from paper_2510_11400_b200 import api, build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU fallback")
    torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", "0")))
    build.build()
    api.lib()
    mode = {"auto": api.FH_SALIENT_AUTO, "off": api.FH_SALIENT_OFF, "all": api.FH_SALIENT_ALL,
            "channel": api.FH_SALIENT_CHANNEL, "tensor": api.FH_SALIENT_TENSOR}[args.mode]
    p = api.default_params(bits=2, salient_mode=mode, rounding=args.rounding, seed=2510_11400)
    items, need = [], 0
    for i, s in enumerate(specs):
        raw = synth.make(s)
        t = torch.from_numpy(raw.view(np.int16) if raw.dtype == np.uint16 else raw).cuda()
        d = api.desc(s.shape, s.dtype, tensor_id=i)
        items.append(api.SchedItem(d, api.FH_COMPRESS if s.compress else api.FH_KEEP, t, torch.empty_like(t)))
        if s.compress:
            need += (api.compressed_bytes(d, p, 1) + 255) & ~255
    arena = torch.empty(need, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(torch.cuda.current_device())
    for _ in range(max(3, args.warmup)):
        rep = api.fh_run_schedule(items, p, arena)
        assert rep.status == api.FH_OK, rep.status
    launches0 = api.kernel_launches()
    sampler.start()
    fwd = bwd = 0.0
    for _ in range(args.steps):
        rep = api.fh_run_schedule(items, p, arena)
        assert rep.status == api.FH_OK, rep.status
        fwd += rep.ms_forward
        bwd += rep.ms_backward
    clocks = sampler.stop()
    launches = api.kernel_launches() - launches0
    dense = int(rep.total_dense_bytes)
    ms = (fwd + bwd) / args.steps
    peak, peak_kind = peaks()
    line = {"metric": METRIC, "value": 2 * dense / (ms / 1e3) / 1e9, "unit": UNIT, "n_gpus": 1, "steps": args.steps,
            "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f32" if specs[0].dtype == synth.F32 else "bf16", "data": "synthetic",
            "config": {"workload": wl_desc + "; through fh_run_schedule, tensors with even index compressed, the rest kept",
                       "bits": [2], "salient_mode": args.mode.upper(), "tensors": len(specs),
                       "compressed_tensors": sum(1 for s in specs if s.compress)},
            "schedule": {"ms_forward": fwd / args.steps, "ms_backward": bwd / args.steps, "total_dense_bytes": dense,
                         "total_packed_bytes": int(rep.total_packed_bytes), "peak_packed_bytes": int(rep.peak_packed_bytes),
                         "compress_gbs": dense / (fwd / args.steps) / 1e6, "decompress_gbs": dense / (bwd / args.steps) / 1e6},
            "roofline": {"bound": "hbm", "kernel": "forward phase: every compress call of the schedule",
                         "achieved": (dense + int(rep.total_packed_bytes)) / (fwd / args.steps) / 1e6, "peak": peak,
                         "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                         "frac": (dense + int(rep.total_packed_bytes)) / (fwd / args.steps) / 1e6 / peak, "traffic": None},
            "clocks": clocks, "gpu_launches": int(launches)}
    print(json.dumps(line), flush=True)
    api.shutdown()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18_b64")
    ap.add_argument("--mode", default="auto", choices=["auto", "off", "all", "channel", "tensor"])
    ap.add_argument("--rounding", type=int, default=0, choices=[0, 1],
                    help="1: random rounding of normal planes (Philox-4x32-10 draws)")
    ap.add_argument("--schedule", action="store_true",
                    help="run the workload through fh_run_schedule (forward-order compress, reverse-order decompress)")
    ap.add_argument("--no-cpu", action="store_true", help="skip the CPU-oracle baseline leg")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer end-to-end leg")
    ap.add_argument("--no-clock-window", action="store_true",
                    help="do not repeat the step (untimed) around the timed region for the clock samples: for runs under a profiler")
    ap.add_argument("--no-sweep", action="store_true", help="skip the size sweep and the schedule leg of the default workload")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    specs, wl_desc = workload_specs(args.workload)
    if args.impl == "reference":
        run_reference(args, specs, wl_desc)
    elif args.schedule:
        run_schedule(args, specs, wl_desc)
    else:
        run_ours(args, specs, wl_desc)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the CacheCard create + inject path.

One *step* is one pass of the whole path over one synthetic cache: offset scan, fused
quantise-pack (create), then unpack-dequantise-scatter (inject).  The default workload is the
Llama-3.1-8B-shaped cache at 8K context with uniform 4-bit tokens; the metric is GB/s of FP16
KV bytes carried through create + inject (KV bytes / (create time + inject time)).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 2|3|4|5] [--impl ours|reference]

With N > 1 (under torchrun) every rank runs an independent replica of the same workload: the
path has no exchange step, so there is no data-path collective.  Rank 0 prints one JSON line.
`--impl reference` times the CPU oracle on the host cores instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2605_03884_b200 import workloads as wl  # noqa: E402

METRIC = "CacheCard create+inject GB/s (FP16 KV bytes) and % of HBM peak at 8K ctx"
UNIT = "GB/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, an earlier measurement of the same copy)"


# what create_kernel and inject_kernel are compiled from
TRAFFIC_SOURCES = ("qkvs_common.cuh", "qkvs_pipeline.cuh", "qkvs_ptx.cuh")


def captured_traffic(kernel: str, n_layers: int):
    """DRAM bytes of one launch of `kernel` at `n_layers` layers, from the committed ncu captures
    of the 8- and the 16-layer case of the headline workload: reads and writes are each taken as
    a straight line through the two captures (reads grow in proportion to the rows; writes too,
    less the lines still dirty in the 126 MB L2 when the kernel ends, which is a constant, not a
    share).  Returns (bytes, how) or (None, why) when the kernels' sources have changed since."""
    import hashlib
    path = os.path.join(ROOT, "profiles", "dram_traffic_llama8b_8k_uniform4.txt")
    csrc = os.path.join(ROOT, "paper_2605_03884_b200", "csrc")
    try:
        entries = {}
        for line in open(path):
            if line.strip() and not line.startswith("#"):
                parts = line.split()
                entries[parts[0]] = parts[1:]
        h = hashlib.sha256()
        for f in TRAFFIC_SOURCES:
            h.update(open(os.path.join(csrc, f), "rb").read())
        if entries.get("csrc_sha256", [""])[0] != h.hexdigest():
            return None, "kernel sources changed since the counters were taken"
        pts = {}
        for key, vals in entries.items():
            if key.startswith(kernel + "@"):
                pts[int(key.split("@")[1])] = (int(vals[0]), int(vals[1]))  # layers -> (read, write)
        (l0, (r0, w0)), (l1, (r1, w1)) = sorted(pts.items())[:2]
        rd = r0 + (r1 - r0) * (n_layers - l0) / (l1 - l0)
        wr = w0 + (w1 - w0) * (n_layers - l0) / (l1 - l0)
        return int(round(rd + wr)), (f"dram__bytes_read.sum and dram__bytes_write.sum captured at {l0} and {l1} layers, "
                                     f"each extended linearly to {n_layers} layers")
    except Exception as e:  # missing or unreadable summary
        return None, f"no usable capture ({type(e).__name__})"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples; summarised over a wall-clock window so that
    only samples taken while the timed work ran count."""

    QUERY = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu_index = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-i", str(self.gpu_index), "-lms", "20"],
                stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self, t_begin: float, t_end: float):
        """Summary of the samples whose timestamp lies in [t_begin, t_end] (time.time() values)."""
        import datetime
        out = {"sm_mhz": None, "sm_max_mhz": None, "power_w_max": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 10:
                        continue
                    try:
                        ts = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                        rows.append((ts, float(parts[2]), float(parts[3]), float(parts[4]),
                                     [n for n, v in zip(names, parts[6:10]) if v.lower().startswith("active")]))
                    except ValueError:
                        continue
            os.unlink(self.path)
        except Exception:
            pass
        inside = [r for r in rows if t_begin - 0.02 <= r[0] <= t_end + 0.02]
        if inside:
            reasons = set()
            for r in inside:
                reasons.update(r[4])
            out.update(sm_mhz=statistics.median(r[1] for r in inside), sm_max_mhz=max(r[2] for r in inside),
                       power_w_max=max(r[3] for r in inside), reasons=sorted(reasons), samples=len(inside))
        return out


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks of the default process group
    (the list itself when there is no group): a replica job is as slow as its slowest rank."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(v) for v in values]
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.tolist()]


def replica_throughput(kv_bytes: int, hops: int, world: int, ms_per_step: float) -> float:
    """Whole-job GB/s of FP16 KV: every rank carries its own cache through create + inject."""
    return kv_bytes * hops * world / (ms_per_step * 1e-3) / 1e9


def load_workload(number: int, layers=None, n_layers=None):
    w = wl.WORKLOADS[number]
    if n_layers:
        w = w.scaled(n_layers=n_layers)   # reduced case for profiler captures only
    Ks, Vs = [], []
    for _, k, v in wl.kv_layers(w, layers):
        Ks.append(k)
        Vs.append(v)
    return w, Ks, Vs


def oracle_rank_rule(scores, n16, n8, n4):
    import oracle
    st, bits = oracle.bits_from_scores(scores, n16, n8, n4)
    assert st == 0
    return bits


def cpu_oracle_leg(w, Ks, Vs, bits, n_layers_sample: int, meta_bytes: int = 8, repeats: int = 3,
                   single_thread_layers: int = 2):
    """Times the oracle as it stands on the first `n_layers_sample` layers: card creation and
    injection each best of `repeats`, the card buffer and the output arrays allocated before the
    clock starts, once with OpenMP over the streams on all host cores and once on a single thread
    (on `single_thread_layers` layers, so that it stays a matter of seconds)."""
    import oracle

    def best_of(L, threads):
        oracle.set_num_threads(threads)
        lay = oracle.make_layout(L, w.n_kv_heads, w.head_dim, w.n_tokens, meta_bytes=meta_bytes)
        st, size = oracle.card_size(lay, bits)
        assert st == 0
        card = np.zeros(size, dtype=np.uint8)
        Ko = [np.zeros_like(k) for k in Ks[:L]]
        Vo = [np.zeros_like(v) for v in Vs[:L]]
        tc, ti = [], []
        for _ in range(repeats):
            t0 = time.perf_counter()
            st1 = oracle.card_create_into(lay, Ks[:L], Vs[:L], bits, card)
            t1 = time.perf_counter()
            st2 = oracle.card_inject(card, lay, Ko, Vo)
            t2 = time.perf_counter()
            assert st1 == 0 and st2 == 0
            tc.append(t1 - t0)
            ti.append(t2 - t1)
        kv = 2 * L * w.n_kv_heads * w.n_tokens * w.head_dim * 2
        return kv, min(tc), min(ti), sum(tc) + sum(ti)

    cores = oracle.num_threads()
    L = min(n_layers_sample, w.n_layers)
    kv, c, i, spent = best_of(L, cores)
    L1 = min(single_thread_layers, L)
    kv1, c1, i1, spent1 = best_of(L1, 1)
    oracle.set_num_threads(cores)
    return {
        "value": kv / (c + i) / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
        "sample": f"layers 0..{L - 1} of the workload ({kv} FP16 KV bytes): create and inject each best of "
                  f"{repeats}, buffers allocated beforehand, OpenMP over streams",
        "create_gbs": kv / c / 1e9, "inject_gbs": kv / i / 1e9,
        "single_thread": {"value": kv1 / (c1 + i1) / 1e9, "create_gbs": kv1 / c1 / 1e9, "inject_gbs": kv1 / i1 / 1e9,
                          "sample": f"layers 0..{L1 - 1} ({kv1} FP16 KV bytes), best of {repeats}, one thread"},
        "seconds": spent + spent1,
    }


def run_reference(args):
    """`--impl reference`: the CPU oracle on the host cores, a bounded sample of the workload per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    sample_layers = 4
    w, Ks, Vs = load_workload(args.config, range(sample_layers))
    bits = wl.bits_for(w, rank_rule=oracle_rank_rule)
    lay = oracle.make_layout(sample_layers, w.n_kv_heads, w.head_dim, w.n_tokens, meta_bytes=args.meta_bytes)
    st, size = oracle.card_size(lay, bits)
    assert st == 0
    card = np.zeros(size, dtype=np.uint8)
    Ko = [np.zeros_like(k) for k in Ks]
    Vo = [np.zeros_like(v) for v in Vs]

    def step():
        assert oracle.card_create_into(lay, Ks, Vs, bits, card) == 0
        assert oracle.card_inject(card, lay, Ko, Vo) == 0

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    kv_bytes = 2 * sample_layers * w.n_kv_heads * w.n_tokens * w.head_dim * 2
    value = kv_bytes * args.steps / dt / 1e9
    sample = (f"layers 0..{sample_layers - 1} of the workload ({kv_bytes} FP16 KV bytes) per step, create then inject, "
              f"buffers allocated beforehand, OpenMP over streams")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "config": {"workload": w.name, "sample_layers": sample_layers,
                                        "meta_bytes_per_group": args.meta_bytes},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


class Case:
    """One workload resident on the device: inputs, outputs, card buffer, scratch block."""

    def __init__(self, q, torch, number, meta_bytes=8, bits_mode=0, n_layers=0, pinned=False, host=None, group_size=32):
        self.q, self.torch = q, torch
        self.number, self.meta_bytes, self.bits_mode, self.group_size = number, meta_bytes, bits_mode, group_size
        w, Ks, Vs = host if host is not None else load_workload(number, n_layers=n_layers)
        self.w, self.Ks, self.Vs = w, Ks, Vs
        self.L, self.H, self.d, self.T = w.n_layers, w.n_kv_heads, w.head_dim, w.n_tokens
        self.hops = w.hops

        def gpu_rank_rule(scores, n16, n8, n4):
            # the adaptive recipe's bit-widths come from the library's own rank kernel
            sd = torch.from_numpy(np.ascontiguousarray(scores, dtype=np.float32)).cuda()
            bd = torch.zeros(scores.size, dtype=torch.uint8, device="cuda")
            q.bits_from_scores(sd, n16, n8, n4, bd)
            torch.cuda.synchronize()
            return bd.cpu().numpy()

        if bits_mode == 1:
            self.bits_per_hop = [wl.bits_per_head(w, h, gpu_rank_rule) for h in range(self.hops)]
        else:
            self.bits_per_hop = [wl.bits_for(w, h, rank_rule=gpu_rank_rule) for h in range(self.hops)]
        self.lay = q.make_layout(self.L, self.H, self.d, self.T, bits_mode=bits_mode, meta_bytes=meta_bytes, group_size=group_size)
        self.sizes = [q.card_size(self.lay, b) for b in self.bits_per_hop]
        self.prefix = q.card_prefix_size(self.lay)
        self.kv_bytes = w.kv_bytes
        if pinned:
            self.Kh = [torch.from_numpy(k).pin_memory() for k in Ks]
            self.Vh = [torch.from_numpy(v).pin_memory() for v in Vs]
            self.bits_h = [torch.from_numpy(b).pin_memory() for b in self.bits_per_hop]
        else:
            self.Kh = [torch.from_numpy(k) for k in Ks]
            self.Vh = [torch.from_numpy(v) for v in Vs]
            self.bits_h = [torch.from_numpy(b) for b in self.bits_per_hop]
        self.Kd = [k.cuda() for k in self.Kh]
        self.Vd = [v.cuda() for v in self.Vh]
        self.Ko = [torch.empty_like(k) for k in self.Kd]
        self.Vo = [torch.empty_like(v) for v in self.Vd]
        self.bits_d = [b.cuda() for b in self.bits_h]
        self.card = torch.zeros(max(self.sizes), dtype=torch.uint8, device="cuda")
        self.ws = q.new_workspace()

    def run_path(self, src_k, src_v, out_k, out_v, bits_dev, on_stream, record=None):
        """create -> inject for every hop of the workload (one hop except for the chain)."""
        q, torch = self.q, self.torch
        for h in range(self.hops):
            if record is not None:
                e0 = torch.cuda.Event(enable_timing=True)
                e1 = torch.cuda.Event(enable_timing=True)
                e2 = torch.cuda.Event(enable_timing=True)
                e0.record(on_stream)
            q.card_create(self.lay, src_k, src_v, bits_dev[h], self.card, card_capacity=self.sizes[h], workspace=self.ws, stream=on_stream)
            if record is not None:
                e1.record(on_stream)
            q.card_inject(self.card, self.lay, out_k, out_v, card_bytes=self.sizes[h], workspace=self.ws, stream=on_stream)
            if record is not None:
                e2.record(on_stream)
                record.append((h, e0, e1, e2))
            src_k, src_v = out_k, out_v  # the next hop re-quantises this hop's output

    def one_step(self, stream, record=None):
        self.run_path(self.Kd, self.Vd, self.Ko, self.Vo, self.bits_d, stream, record)

    def timed(self, stream, steps, warmup, barrier=None):
        """`warmup` untimed steps, then exactly `steps` timed ones between two synchronisations.
        Returns (total ms, per-hop create ms lists, per-hop inject ms lists)."""
        torch = self.torch
        for _ in range(warmup):
            self.one_step(stream)
        torch.cuda.synchronize()
        st, _ = self.q.card_info(self.card)
        if st != 0:
            raise RuntimeError(f"card status {st}")
        if barrier:
            barrier()
        torch.cuda.synchronize()
        records = []
        t_begin = torch.cuda.Event(enable_timing=True)
        t_end = torch.cuda.Event(enable_timing=True)
        t_begin.record(stream)
        for _ in range(steps):
            self.one_step(stream, records)
        t_end.record(stream)
        torch.cuda.synchronize()
        if barrier:
            barrier()
        create_ms = [[] for _ in range(self.hops)]
        inject_ms = [[] for _ in range(self.hops)]
        for h, e0, e1, e2 in records:
            create_ms[h].append(e0.elapsed_time(e1))
            inject_ms[h].append(e1.elapsed_time(e2))
        return t_begin.elapsed_time(t_end), create_ms, inject_ms

    def attend(self, stream, per_kv=4, reps=25):
        """Decode-step attention straight from the card the last create left behind: median ms."""
        q, torch = self.q, self.torch
        n_q = per_kv * self.H
        qd = torch.randn((self.L, n_q, self.d), device="cuda").half()
        od = torch.zeros((self.L, n_q, self.d), dtype=torch.float32, device="cuda")
        scratch = torch.zeros(q.attend_scratch_size(self.lay, n_q), dtype=torch.uint8, device="cuda")
        ev = []
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            q.card_attend(self.card, self.lay, qd, od, scratch, card_bytes=self.sizes[-1], stream=stream)
            b.record(stream)
            ev.append((a, b))
        torch.cuda.synchronize()
        if int(scratch[:4].view(torch.int32).item()) != 0:
            raise RuntimeError("attention from the card reported a bad card")
        return statistics.median(x.elapsed_time(y) for x, y in ev[5:])

    def hop_stats(self, create_ms, inject_ms, peak, errors=None):
        med = statistics.median
        out = []
        for h in range(self.hops):
            payload = self.sizes[h] - self.prefix
            c, i = med(create_ms[h]), med(inject_ms[h])
            moved = self.kv_bytes + payload
            entry = {
                "hop": h, "card_bytes": self.sizes[h],
                "avg_code_bits": float(self.bits_per_hop[h].astype(np.float64).mean()),
                "create_ms": c, "inject_ms": i, "create_ms_min": min(create_ms[h]), "inject_ms_min": min(inject_ms[h]),
                "create_kv_gbs": self.kv_bytes / (c * 1e-3) / 1e9, "inject_kv_gbs": self.kv_bytes / (i * 1e-3) / 1e9,
                "create_hbm_frac": moved / (c * 1e-3) / 1e9 / peak, "inject_hbm_frac": moved / (i * 1e-3) / 1e9 / peak,
            }
            if errors is not None:
                entry["error_vs_original"] = errors[h]
            out.append(entry)
        return out

    def errors(self, stream):
        """What the handoff costs in accuracy: every hop's injected cache against the original FP16
        cache (reporting only, outside every timed region; plain torch reductions)."""
        q, torch = self.q, self.torch

        def error_of(out, ref):
            mx, se, sr = 0.0, 0.0, 0.0
            for o, r in zip(out, ref):
                dlt = o.float() - r.float()
                mx = max(mx, float(dlt.abs().max()))
                se += float(dlt.double().pow(2).sum())
                sr += float(r.double().pow(2).sum())
            n = sum(r.numel() for r in ref)
            return {"max_abs": mx, "rmse": (se / n) ** 0.5, "rel_frobenius": (se / sr) ** 0.5 if sr else 0.0}

        res = []
        src_k, src_v = self.Kd, self.Vd
        for h in range(self.hops):
            q.card_create(self.lay, src_k, src_v, self.bits_d[h], self.card, card_capacity=self.sizes[h], workspace=self.ws, stream=stream)
            q.card_inject(self.card, self.lay, self.Ko, self.Vo, card_bytes=self.sizes[h], workspace=self.ws, stream=stream)
            torch.cuda.synchronize()
            res.append({"K": error_of(self.Ko, self.Kd), "V": error_of(self.Vo, self.Vd)})
            src_k, src_v = self.Ko, self.Vo
        return res


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2605_03884_b200 as q
    from paper_2605_03884_b200 import build as qbuild

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    if rank == 0:
        qbuild.build()
    if world > 1:
        dist.barrier()
    q.load_library()
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()  # runs through set-up and both timed legs; summarised over the timed window

    case = Case(q, torch, args.config, args.meta_bytes, args.bits_mode, args.layers, pinned=not args.skip_e2e, group_size=args.group_size)
    w, L, H, d, T, hops = case.w, case.L, case.H, case.d, case.T, case.hops
    kv_bytes, sizes, prefix = case.kv_bytes, case.sizes, case.prefix
    Kd, Vd, Ko, Vo, Kh, Vh, bits_d, bits_h = case.Kd, case.Vd, case.Ko, case.Vo, case.Kh, case.Vh, case.bits_d, case.bits_h
    stream = torch.cuda.current_stream()
    barrier = dist.barrier if world > 1 else None

    t_wall_begin = time.time()
    total_ms, create_ms, inject_ms = case.timed(stream, args.steps, max(args.warmup, 3), barrier)

    # end-to-end leg: host buffers in, host buffers out, copies inside the timed region
    e2e_ms = e2e_serial_ms = float("nan")
    if not args.skip_e2e:
        Koh = [torch.empty_like(k).pin_memory() for k in Kh]
        Voh = [torch.empty_like(v).pin_memory() for v in Vh]

        def e2e_serial_step():
            for dst, src in zip(Kd + Vd, Kh + Vh):
                dst.copy_(src, non_blocking=True)
            for bd, bh in zip(bits_d, bits_h):
                bd.copy_(bh, non_blocking=True)
            case.one_step(stream)
            for dst, src in zip(Koh + Voh, Ko + Vo):
                dst.copy_(src, non_blocking=True)

        def e2e_pipelined(n_steps):
            """Host buffers in, host buffers out, every step: the copy-in of step i+1, the kernels of
            step i and the copy-out of step i-1 run on three streams over two sets of device
            buffers.  Returns the device time from the first copy-in to the last copy-out (ms)."""
            s_in, s_cmp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
            sets = [dict(K=Kd, V=Vd, Ko=Ko, Vo=Vo, bits=bits_d),
                    dict(K=[torch.empty_like(t) for t in Kd], V=[torch.empty_like(t) for t in Vd],
                         Ko=[torch.empty_like(t) for t in Ko], Vo=[torch.empty_like(t) for t in Vo],
                         bits=[torch.empty_like(t) for t in bits_d])]
            torch.cuda.synchronize()
            e_begin = torch.cuda.Event(enable_timing=True)
            e_end = torch.cuda.Event(enable_timing=True)
            ev_cmp, ev_out = [], []
            e_begin.record(s_in)
            for i in range(n_steps):
                b = sets[i % 2]
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_cmp[i - 2])   # the kernels of step i-2 have read these inputs
                    for dst, src in zip(b["K"] + b["V"], Kh + Vh):
                        dst.copy_(src, non_blocking=True)
                    for bd, bh in zip(b["bits"], bits_h):
                        bd.copy_(bh, non_blocking=True)
                    ev_in = torch.cuda.Event()
                    ev_in.record(s_in)
                with torch.cuda.stream(s_cmp):
                    s_cmp.wait_event(ev_in)
                    if i >= 2:
                        s_cmp.wait_event(ev_out[i - 2])  # the copy-out of step i-2 has drained these outputs
                    case.run_path(b["K"], b["V"], b["Ko"], b["Vo"], b["bits"], s_cmp)
                    ev = torch.cuda.Event()
                    ev.record(s_cmp)
                    ev_cmp.append(ev)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_cmp[i])
                    for dst, src in zip(Koh + Voh, b["Ko"] + b["Vo"]):
                        dst.copy_(src, non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(s_out)
                    ev_out.append(ev)
            e_end.record(s_out)
            torch.cuda.synchronize()
            return e_begin.elapsed_time(e_end)

        e2e_serial_step()
        torch.cuda.synchronize()
        n_serial = max(3, min(args.steps, 20))
        e_begin = torch.cuda.Event(enable_timing=True)
        e_end = torch.cuda.Event(enable_timing=True)
        e_begin.record(stream)
        for _ in range(n_serial):
            e2e_serial_step()
        e_end.record(stream)
        torch.cuda.synchronize()
        e2e_serial_ms = e_begin.elapsed_time(e_end) / n_serial
        e2e_pipelined(3)
        if world > 1:
            dist.barrier()
        e2e_ms = e2e_pipelined(args.steps)
        del Koh, Voh
    torch.cuda.synchronize()
    clocks = sampler.stop(t_wall_begin, time.time()) if rank == 0 else None

    peak, peak_src = measured_peaks()

    # attention straight from the card (the row after the hot path): one decode step, 32 query
    # heads, over the card the last create left behind; reported beside the main metric
    attend = None
    if d == 128 and not args.skip_attend:
        a_ms = case.attend(stream, 4)
        payload = sizes[-1] - prefix
        attend = {"what": "decode-step attention straight from the card, all layers, 4 query heads per KV head",
                  "ms": a_ms, "card_payload_bytes": payload, "card_gbs": payload / (a_ms * 1e-3) / 1e9,
                  "hbm_frac": payload / (a_ms * 1e-3) / 1e9 / peak,
                  # eight query rows per KV head fill the products' columns: two new tokens of a 4:1
                  # grouped-query model (their heads laid out as eight heads per KV head) in one pass
                  "ms_8_rows_per_kv_head": case.attend(stream, 8)}

    hop_errors = case.errors(stream) if rank == 0 else None
    total_ms, e2e_ms = max_over_ranks([total_ms, e2e_ms], device="cuda")

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    ms_per_step = total_ms / args.steps
    value = replica_throughput(kv_bytes, hops, world, ms_per_step)
    e2e_value = None if args.skip_e2e else replica_throughput(kv_bytes, hops, world, e2e_ms / args.steps)
    per_hop = case.hop_stats(create_ms, inject_ms, peak, hop_errors)
    # dominant kernel: the slower of the two halves on hop 0
    payload0 = sizes[0] - prefix
    c0 = sum(create_ms[0]) / len(create_ms[0])
    i0 = sum(inject_ms[0]) / len(inject_ms[0])
    if c0 >= i0:
        dom, dom_ms, dom_key = "create_kernel (timed together with the offset scan that precedes it)", c0, "create_kernel"
    else:
        dom, dom_ms, dom_key = "inject_kernel", i0, "inject_kernel"
    achieved = (kv_bytes + payload0) / (dom_ms * 1e-3) / 1e9
    if w.number == 3 and args.meta_bytes == 8 and args.bits_mode == 0:
        traffic, traffic_how = captured_traffic(dom_key, L)
    else:
        traffic, traffic_how = None, "captured for the headline workload only"
    roofline = {"bound": "hbm", "kernel": dom, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_source": peak_src, "traffic": traffic, "traffic_how": traffic_how,
                "algorithmic_bytes_per_launch": kv_bytes + payload0, "avg_launch_ms": dom_ms,
                "datasheet_peak": 8000.0, "frac_of_datasheet": achieved / 8000.0}

    # per hop: the offset scan (plus its second stage with per-head bit-widths), then one create
    # and one inject launch per block of 64 layers
    launches_per_step = hops * (1 + args.bits_mode + 2 * ((L + 63) // 64))
    cpu = None
    if not args.no_cpu_baseline:
        cpu = cpu_oracle_leg(w, case.Ks, case.Vs, case.bits_per_hop[0][:T], L, args.meta_bytes)

    # the step in front of the path: bit-widths from importance scores (config 4's recipe by rank;
    # the same under a byte budget of 100 bytes per token, with the offset table from the same
    # launch), at the workload's length and at 128K tokens
    rank_us = None
    bits_rules = None
    if not args.skip_attend:
        def timed_us(fn, reps):
            for _ in range(5):
                fn()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for _ in range(reps):  # back to back: one call alone would time the host's launch latency
                fn()
            b.record(stream)
            torch.cuda.synchronize()
            return a.elapsed_time(b) * 1e3 / reps

        bits_rules = {}
        for n_tok, reps in ((T, 50), (131072, 10)):
            sc = torch.randn(n_tok, device="cuda").exp()
            bd = torch.zeros(n_tok, dtype=torch.uint8, device="cuda")
            od = torch.zeros(n_tok + 1, dtype=torch.int32, device="cuda")
            c16, c8, c4 = wl.quantile_counts(n_tok)
            by_rank = timed_us(lambda: q.bits_from_scores(sc, c16, c8, c4, bd, stream=stream), reps)
            by_budget = timed_us(lambda: q.bits_from_scores_budget(sc, d, 100 * n_tok, bd, meta_bytes=args.meta_bytes,
                                                                   offsets_dev=od, stream=stream), reps)
            bits_rules[str(n_tok)] = {"by_rank_us": by_rank, "by_budget_with_offsets_us": by_budget}
            if n_tok == T:
                rank_us = by_rank
            del sc, bd, od

    # the other benchmark workloads and card formats, a few steps each, after the headline timing
    # and outside it: the 1K mixed cache, the 8K adaptive cache, the four-hop chain; then the 8K
    # uniform and adaptive caches with FP16 scale/zero pairs and with groups of 64 and 128 channels
    # (these with the reconstruction error of the injected cache against the original)
    per_config = None
    if args.per_config and w.number == 3 and not args.layers and args.meta_bytes == 8 and args.bits_mode == 0 and args.group_size == 32:
        per_config = []
        hosts = {3: (case.w, case.Ks, case.Vs)}
        del case, Kd, Vd, Ko, Vo, Kh, Vh, bits_d, bits_h
        torch.cuda.empty_cache()
        runs = ((2, 8, 32), (4, 8, 32), (5, 8, 32), (3, 4, 32), (4, 4, 32), (3, 8, 64), (4, 8, 64), (3, 4, 128), (4, 4, 128))
        for number, meta, group in runs:
            src = 3 if number == 5 else number      # the chain starts from the headline cache; same bytes
            if src not in hosts and src != 2:
                hosts[src] = load_workload(src)
            hw = (wl.WORKLOADS[number], hosts[src][1], hosts[src][2]) if src in hosts else None
            c = Case(q, torch, number, meta, 0, 0, pinned=False, host=hw, group_size=group)
            _, cm, im = c.timed(stream, args.per_config_steps, 3)
            errs = c.errors(stream) if (meta, group) != (8, 32) else None
            entry = {"workload": c.w.name, "meta_bytes_per_group": meta, "group_size": group, "steps": args.per_config_steps,
                     "fp16_kv_bytes": c.kv_bytes,
                     "bits_per_element": 8.0 * (c.sizes[0] - c.prefix) / (c.kv_bytes / 2),
                     "per_hop": c.hop_stats(cm, im, peak, errs)}
            if c.d == 128 and not args.skip_attend:
                a_ms = c.attend(stream, 4, reps=15)
                payload = c.sizes[-1] - c.prefix
                entry["attend_from_card"] = {"ms": a_ms, "card_payload_bytes": payload,
                                             "hbm_frac": payload / (a_ms * 1e-3) / 1e9 / peak}
            per_config.append(entry)
            del c
            torch.cuda.empty_cache()

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name, "n_layers": L, "n_kv_heads": H, "head_dim": d, "n_tokens": T,
                   "hops": hops, "fp16_kv_bytes": kv_bytes, "replicas": world,
                   "meta_bytes_per_group": args.meta_bytes, "group_size": args.group_size, "bits_mode": args.bits_mode,
                   "reduced_for_profiling": bool(args.layers),
                   "l2": "inputs (1 GiB FP16 KV per pass) exceed the 126 MB L2; no flush"
                   if kv_bytes > 4 * 126e6 else "working set comparable to L2; L2 helps"},
        "per_hop": per_hop,
        "roofline": roofline,
        "cpu_baseline": cpu,
        "e2e": {"value": e2e_value, "unit": UNIT,
                "h2d_bytes_per_step": kv_bytes + hops * T * (L * H if args.bits_mode == 1 else 1),
                "d2h_bytes_per_step": kv_bytes,
                "ms_per_step": None if args.skip_e2e else e2e_ms / args.steps,
                "how": "pinned host buffers in and out every step; copy-in, kernels and copy-out of "
                       "neighbouring steps overlap on three streams over two sets of device buffers",
                "serial_ms_per_step": None if args.skip_e2e else e2e_serial_ms},
        "gpu_launches": launches_per_step * args.steps,
        "clocks": clocks,
        "attend_from_card": attend,
        "bits_from_scores_us": rank_us,
        "bits_from_scores": bits_rules,
        "per_config": per_config,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=3, choices=[2, 3, 4, 5])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--skip-e2e", action="store_true", help="skip the host-buffer leg (profiler captures)")
    ap.add_argument("--skip-attend", action="store_true", help="skip the attention-from-the-card measurement")
    ap.add_argument("--no-per-config", dest="per_config", action="store_false",
                    help="skip the short runs of the other benchmark workloads after the headline")
    ap.add_argument("--per-config-steps", type=int, default=10)
    ap.add_argument("--meta-bytes", type=int, default=8, choices=[8, 4],
                    help="bytes of scale and zero per group in the card: 8 = two fp32 (the headline format), "
                         "4 = two FP16 (compact variant)")
    ap.add_argument("--group-size", type=int, default=32, choices=[32, 64, 128],
                    help="channels per quantisation group (32 is the headline format)")
    ap.add_argument("--bits-mode", type=int, default=0, choices=[0, 1],
                    help="0: one bit-width vector for the whole model (the paper's); 1: one per (layer, KV head)")
    ap.add_argument("--layers", type=int, default=0,
                    help="reduced case for profiler captures: keep the workload's recipe at this many layers")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the SWAA attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One step = one pass of the whole hot path over one batch of synthetic input:
    layer schedule (host)  ->  swaa_prefill on the long-context SWA workload (L=32768, Hq=32, Hkv=8,
    D=128, W=2048, n_sink=4)  ->  swaa_decode with full attention ("FA Decode") on the decode workload
    (B=16, 65536-entry cache)  ->  swaa_decode with the SWA mask (n_sink=4 + W=4096 entries).
Each kernel is bracketed by CUDA events on the launching stream; L2 is flushed before each kernel (a
256 MiB write, then a 256 MiB read of another buffer so that the lines left in L2 are clean and their
eviction is not charged to the timed kernel) so every launch reads its inputs from HBM.  `value` is the effective prefill throughput
4*D*Hq*visible_pairs / (prefill kernel time), aggregated over ranks (max time over ranks); decode
bandwidth goes into the `decode` object.  With N > 1 every rank runs the same independent problem
(weak scaling, no collective on the data path).

--impl reference times the float64 CPU oracle (the only "reference" this method has) on a bounded
row sample of the same prefill workload, on the host cores, rank 0 only.
"""
import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "swa_prefill_effective_tflops"
UNIT = "TFLOP/s"
L2_FLUSH_BYTES = 256 << 20

# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under profiles/ (first of
# the two captured launches each; taken on the kernels as committed).
PREFILL_DRAM_TRAFFIC_BYTES = 404582656 + 236282112  # profiles/prefill_kernel_cfg2_long_swa.txt

# FA decode: 4 x the B=4 capture (traffic grows in proportion to B), profiles/decode_kernel_fa_quarter_of_cfg4.txt;
# SWA decode: full size, profiles/decode_kernel_swa_cfg4.txt
DECODE_FA_DRAM_TRAFFIC_BYTES = 4 * (1073863000 + 3872512)
DECODE_SWA_DRAM_TRAFFIC_BYTES = 269665536 + 4531200


def visible_pairs(L, W, S, full):
    if full or W >= L:
        return L * (L + 1) // 2
    if L >= W + S:
        return W * (W + 1) // 2 + (L - W) * W + S * (S + 1) // 2 + (L - W - S) * S
    return sum(min(i + 1, W) + max(0, min(S, i - W + 1)) for i in range(L))


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, uuid: str, period_s: float = 0.02):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._uuid, self._period = uuid, period_s
        try:
            import pynvml

            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode() if isinstance(uuid, str) else uuid)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nv = None

    def _run(self):
        nv = self._nv
        names = {
            "hw_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8),
            "hw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40),
            "sw_thermal_slowdown": getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20),
            "sw_power_cap": getattr(nv, "nvmlClocksThrottleReasonSwPowerCap", 0x4),
            "hw_power_brake": getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80),
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
                for k, bit in names.items():
                    if mask & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(self._period)

    def start(self):
        if self._nv is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()
        s = sorted(self.samples)
        return {"sm_mhz": (s[len(s) // 2] if s else None), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def run_reference(args, rank):
    """The oracle as it stands, on the host cores: each step computes a bounded row sample of the
    long-context SWA prefill workload; throughput is reported in the same unit as the GPU arm."""
    if rank != 0:
        return
    import numpy as np

    import oracle
    from paper_2512_10411_b200 import inputs

    cfg = inputs.cfg_long()
    q, k, v, cu = inputs.make_prefill_inputs(cfg, "cpu")
    qh, kh, vh = (inputs.to_f32_numpy(t) for t in (q, k, v))
    L = cfg.seqlens[0]
    rng = np.random.default_rng(1234)

    def sample(n):
        rt = rng.integers(cfg.window + cfg.n_sink, L, n)  # rows with a full window: S + W visible keys each
        rh = rng.integers(0, cfg.Hq, n).astype(np.int32)
        return rt, rh

    def run(rows):
        t0 = time.perf_counter()
        r = oracle.prefill(qh, kh, vh, [0, L], cfg.window, cfg.n_sink, False, rows=rows)
        dt = time.perf_counter() - t0
        return dt, 4.0 * cfg.D * float(r["nvis"].sum())

    dt, _ = run(sample(256))
    budget = 150.0 / max(1, args.steps + args.warmup)          # whole run within a few minutes
    n_rows = int(max(32, min(65536, 256 * min(budget, 20.0) / max(dt, 1e-6))))
    for _ in range(args.warmup):
        run(sample(n_rows))
    total_t, total_f = 0.0, 0.0
    for _ in range(args.steps):
        dt, fl = run(sample(n_rows))
        total_t += dt
        total_f += fl
    value = total_f / total_t / 1e12
    cores = oracle.num_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_t / max(1, args.steps), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "cfg2 long-context SWA prefill: B=1 L=32768 Hq=32 Hkv=8 D=128 W=2048 n_sink=4",
                   "sample": f"{n_rows} seeded (row, head) rows per step"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{n_rows} seeded (row, head) rows per step, {args.steps} steps"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def max_over_ranks(values, world, device=None):
    """Every rank runs the same independent problem (replicas, no collective on the data path); a timing of
    the job is the slowest rank's.  Returns the element-wise maximum over ranks of `values` on every rank."""
    import torch

    t = torch.tensor(values, dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist

        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def stats_ms(values):
    """median / min / mean of a list of per-launch times (ms)."""
    v = sorted(values)
    n = len(v)
    med = v[n // 2] if n % 2 else 0.5 * (v[n // 2 - 1] + v[n // 2])
    return {"median": med, "min": v[0], "mean": sum(v) / n, "n": n}


def time_prefill_case(swaa, torch, flush_l2, stream, peaks, cfg, is_full, reps, tensors=None, sustained=False):
    """One swaa_prefill workload: `reps` timed launches after one warm-up, L2 flushed before each, CUDA events
    on the launching stream.  Returns a dict with median / min time and effective throughput."""
    from paper_2512_10411_b200 import inputs

    q, k, v, cu = tensors if tensors is not None else inputs.make_prefill_inputs(cfg, "cuda")
    out = torch.empty_like(q)
    ms = []
    for r in range(reps + 1):
        flush_l2()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        swaa.swaa_prefill(q, k, v, out, cu, max(cfg.seqlens), cfg.window, cfg.n_sink, is_full)
        b.record(stream)
        torch.cuda.synchronize()
        if r > 0:
            ms.append(a.elapsed_time(b))
    if swaa.last_device_status() != 0:
        raise RuntimeError("swaa_prefill reported a device error")
    st = stats_ms(ms)
    pairs = sum(visible_pairs(L, cfg.window, cfg.n_sink, is_full) for L in cfg.seqlens)
    flops = 4.0 * cfg.D * cfg.Hq * pairs
    tf = flops / (st["median"] * 1e-3) / 1e12
    peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    del out
    return {"seqlens": list(cfg.seqlens) if len(cfg.seqlens) > 1 else cfg.seqlens[0], "Hq": cfg.Hq, "Hkv": cfg.Hkv,
            "D": cfg.D, "window": cfg.window, "n_sink": cfg.n_sink, "is_full": bool(is_full), "ms": st["median"],
            "ms_min": st["min"], "launches": st["n"], "effective_tflops": tf, "frac_of_measured_peak": tf / peak,
            "frac_of_nominal_2250": tf / 2250.0, "us_per_1k_tokens": 1e3 * st["median"] / (sum(cfg.seqlens) / 1024.0)}


def gather_decode_partials(part, world):
    """The one exchange of a decode whose cache is cut along the context: every rank contributes its partial
    results [B, Hq, D + 2] (float32) and receives all of them as [world, B, Hq, D + 2], rank-major, ready for
    swaa_decode_combine.  B * Hq * (D + 2) floats per rank (266 KB at workload 4)."""
    import torch

    if world == 1:
        return part.unsqueeze(0).contiguous()
    import torch.distributed as dist

    out = torch.empty((world,) + tuple(part.shape), dtype=part.dtype, device=part.device)
    # concatenation along the first dimension: rank r's partials land in rows [r * B, (r + 1) * B)
    dist.all_gather_into_tensor(out.view((world * part.shape[0],) + tuple(part.shape[1:])), part.contiguous())
    return out


def exchange_halo_and_sinks(k_own, v_own, window, n_sink, rank, world):
    """The data movement of a context-parallel SWA prefill for one sequence cut into `world` equal stretches: rank r
    owns k_own, v_own [L / world, Hkv, D] (positions r * L / world ...).  It receives the last window - 1 rows of rank
    r - 1 (one neighbour send; the stretch must be at least that long) and the first n_sink rows of rank 0 (one
    broadcast).  Returns (k_local, v_local, sink_k, sink_v, key_pos0): halo ++ own stretch, the sink rows as
    [1, max(n_sink, 1), Hkv, D], and the position of the first local key -- the arguments of
    swaa_prefill_context_parallel."""
    import torch
    import torch.distributed as dist

    own = k_own.shape[0]
    halo = min(window - 1, own) if rank > 0 else 0
    if world > 1 and window - 1 > own:
        raise ValueError("the stretch of a rank must hold at least window - 1 tokens")
    sink_rows = max(n_sink, 1)
    sink_k = torch.zeros((1, sink_rows) + tuple(k_own.shape[1:]), dtype=k_own.dtype, device=k_own.device)
    sink_v = torch.zeros_like(sink_k)
    if rank == 0:
        m = min(sink_rows, own)
        sink_k[0, :m] = k_own[:m]
        sink_v[0, :m] = v_own[:m]
    if world == 1:
        return k_own, v_own, sink_k, sink_v, 0
    dist.broadcast(sink_k, src=0)
    dist.broadcast(sink_v, src=0)
    send_rows = min(window - 1, own)
    k_local = torch.empty((halo + own,) + tuple(k_own.shape[1:]), dtype=k_own.dtype, device=k_own.device)
    v_local = torch.empty_like(k_local)
    k_local[halo:] = k_own
    v_local[halo:] = v_own
    ops = []
    if rank + 1 < world:
        ops += [dist.P2POp(dist.isend, k_own[own - send_rows:].contiguous(), rank + 1),
                dist.P2POp(dist.isend, v_own[own - send_rows:].contiguous(), rank + 1)]
    if rank > 0:
        hk = torch.empty((halo,) + tuple(k_own.shape[1:]), dtype=k_own.dtype, device=k_own.device)
        hv = torch.empty_like(hk)
        ops += [dist.P2POp(dist.irecv, hk, rank - 1), dist.P2POp(dist.irecv, hv, rank - 1)]
    if ops:
        for req in dist.batch_isend_irecv(ops):
            req.wait()
    if rank > 0:
        k_local[:halo] = hk
        v_local[:halo] = hv
    return k_local, v_local, sink_k, sink_v, rank * own - halo


def run_context_parallel(args, rank, local_rank, world):
    """Workload 2 (SWA prefill, L=32768) cut along the context over the ranks (strong scaling): halo and sink rows are
    moved by exchange_halo_and_sinks, then every rank runs swaa_prefill_context_parallel on its stretch.  The two parts
    are timed separately; with one rank there is nothing to move."""
    import torch

    import paper_2512_10411_b200 as swaa
    from paper_2512_10411_b200 import inputs

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    cfg = inputs.cfg_long()
    L = cfg.seqlens[0]
    q, k, v, _ = inputs.make_prefill_inputs(cfg, dev)   # every rank draws the same sequence and keeps its stretch
    own = L // world
    sl = slice(rank * own, (rank + 1) * own)
    q_own, k_own, v_own = q[sl].contiguous(), k[sl].contiguous(), v[sl].contiguous()
    del q, k, v
    out = torch.empty_like(q_own)
    cu_q = torch.tensor([0, own], dtype=torch.int32, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    t_x, t_k = [], []
    for it in range(max(args.warmup, 3) + args.steps):
        flush.zero_()
        flush_rd.sum()
        if world > 1:
            dist.barrier()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(stream)
        k_loc, v_loc, sk, sv, p0 = exchange_halo_and_sinks(k_own, v_own, cfg.window, cfg.n_sink, rank, world)
        e[1].record(stream)
        cu_k = torch.tensor([0, k_loc.shape[0]], dtype=torch.int32, device=dev)
        pos0 = torch.tensor([p0], dtype=torch.int32, device=dev)
        swaa.swaa_prefill_context_parallel(q_own, k_loc, v_loc, sk, sv, out, cu_q, cu_k, pos0, own, k_loc.shape[0],
                                           cfg.window, cfg.n_sink)
        e[2].record(stream)
        torch.cuda.synchronize()
        if it >= max(args.warmup, 3):
            t_x.append(e[0].elapsed_time(e[1]))
            t_k.append(e[1].elapsed_time(e[2]))
    assert swaa.last_device_status() == 0
    med_x, med_k = max_over_ranks([stats_ms(t_x)["median"], stats_ms(t_k)["median"]], world, dev)
    flops = 4.0 * cfg.D * cfg.Hq * visible_pairs(L, cfg.window, cfg.n_sink, False)
    if rank == 0:
        tf = flops / ((med_x + med_k) * 1e-3) / 1e12
        print(json.dumps({"metric": METRIC, "value": tf, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                          "warmup": max(args.warmup, 3), "ms_per_step": med_x + med_k, "higher_is_better": True,
                          "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                          "config": {"workload": f"cfg2 long-context SWA prefill cut along the context over {world} rank(s)",
                                     "l2": "flushed before every step"},
                          "context_parallel": {"exchange_ms": med_x, "kernel_ms": med_k,
                                               "kernel_tflops_all_ranks": flops / (med_k * 1e-3) / 1e12,
                                               "frac_of_measured_peak_per_gpu": flops / world / (med_k * 1e-3) / 1e12 / peaks["bf16_tflops"]}}))
    if world > 1:
        dist.destroy_process_group()


def run_decode_split(args, rank, local_rank, world):
    """Decode workload 4 with the cache cut along the context over the ranks (strong scaling: the job is one decode
    step of the whole batch).  Rank r holds positions [r * Lmax / N, (r + 1) * Lmax / N) of every sequence; a step is
    swaa_decode_partial on the shard, the gather of the partials, swaa_decode_combine.  With one rank the shards of an
    N-way cut (--shards) are run one after another on the same GPU, which gives kernel times but no exchange."""
    import torch

    import paper_2512_10411_b200 as swaa
    from paper_2512_10411_b200 import inputs

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    peaks = load_peaks()
    dcfg = inputs.cfg_decode()
    P = world if world > 1 else max(1, args.shards)
    Lsh = dcfg.Lmax // P
    mine = [rank] if world > 1 else list(range(P))
    q, kc, vc, sl = inputs.make_decode_inputs(dcfg, dev)
    shards = [(kc[:, r * Lsh:(r + 1) * Lsh].contiguous(), vc[:, r * Lsh:(r + 1) * Lsh].contiguous(), r * Lsh) for r in mine]
    del kc, vc
    out = torch.empty_like(q)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream()
    results = {}
    for full in (True, False):
        ws = torch.empty(swaa.decode_partial_workspace_size(dcfg.B, dcfg.Hq, dcfg.Hkv, dcfg.D, Lsh, dcfg.window, dcfg.n_sink,
                                                            full), dtype=torch.uint8, device=dev)
        parts = torch.empty((len(mine), dcfg.B, dcfg.Hq, dcfg.D + 2), dtype=torch.float32, device=dev)
        times = []
        for it in range(max(args.warmup, 3) + args.steps):
            flush.zero_()
            flush_rd.sum()
            if world > 1:
                dist.barrier()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i, (ks, vs, p0) in enumerate(shards):
                swaa.swaa_decode_partial(q, ks, vs, parts[i], sl, p0, dcfg.window, dcfg.n_sink, full, ws)
            allp = gather_decode_partials(parts[0], world) if world > 1 else parts
            swaa.swaa_decode_combine(allp, out)
            b.record(stream)
            torch.cuda.synchronize()
            if it >= max(args.warmup, 3):
                times.append(a.elapsed_time(b))
        assert swaa.last_device_status() == 0
        med = max_over_ranks([stats_ms(times)["median"]], world, dev)[0]
        nbytes = float(dcfg.B) * (dcfg.Lmax if full else dcfg.window + dcfg.n_sink) * dcfg.Hkv * dcfg.D * 4
        results["fa" if full else "swa"] = {"us_per_step": 1e3 * med, "gbs": nbytes / (med * 1e-3) / 1e9, "bytes": nbytes}
    if rank == 0:
        print(json.dumps({"metric": "decode_split_hbm_gbs", "value": results["fa"]["gbs"], "unit": "GB/s", "n_gpus": world,
                          "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": results["fa"]["us_per_step"] / 1e3,
                          "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16",
                          "data": "synthetic",
                          "config": {"workload": f"cfg4 decode B=16 Lcache=65536 cut along the context into {P} shards"
                                                 + ("" if world > 1 else " run one after another on one GPU (no exchange)"),
                                     "l2": "flushed before every step"},
                          "decode_split": results, "hbm_peak_gbs": peaks["hbm_gbs"]}))
    if world > 1:
        dist.destroy_process_group()


def whole_job_value(units_per_rank, n_ranks, seconds):
    """Throughput of the whole job: the units all ranks processed over the slowest rank's time."""
    return n_ranks * units_per_rank / seconds


def run_ours(args, rank, local_rank, world):
    import numpy as np
    import torch

    import paper_2512_10411_b200 as swaa
    from paper_2512_10411_b200 import inputs

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        import torch.distributed as dist

        dist.init_process_group("nccl", device_id=dev)
    swaa.load_library()
    peaks = load_peaks()

    # ---------------------------------------------------------------- workloads (resident in HBM)
    pcfg = inputs.cfg_long()
    q, k, v, cu = inputs.make_prefill_inputs(pcfg, dev)
    out = torch.empty_like(q)
    L = pcfg.seqlens[0]
    dcfg = inputs.cfg_decode()
    dq, kc, vc, sl = inputs.make_decode_inputs(dcfg, dev)
    dout = torch.empty_like(dq)
    ws_fa = torch.empty(swaa.decode_workspace_size(dcfg.B, dcfg.Hq, dcfg.Hkv, dcfg.D, dcfg.Lmax, dcfg.window,
                                                   dcfg.n_sink, True), dtype=torch.uint8, device=dev)
    ws_swa = torch.empty(swaa.decode_workspace_size(dcfg.B, dcfg.Hq, dcfg.Hkv, dcfg.D, dcfg.Lmax, dcfg.window,
                                                    dcfg.n_sink, False), dtype=torch.uint8, device=dev)
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    flush_rd = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device=dev)

    def flush_l2():
        flush.zero_()          # displaces everything ...
        flush_rd.sum()         # ... and replaces the dirty lines of that write by clean ones
    # one SWAA recipe: SWA prefill on this layer, FA decode on; and its SWA-decode counterpart
    pol_fa_decode = swaa.SwaaPolicy(n_layers=36, window=pcfg.window, n_sink=pcfg.n_sink, fa_start=3, fa_step=4,
                                    fa_decode=True)
    pol_swa_decode = swaa.SwaaPolicy(n_layers=36, window=dcfg.window, n_sink=dcfg.n_sink, fa_start=3, fa_step=4,
                                     fa_decode=False)
    layer = 0

    prefill_flops = 4.0 * pcfg.D * pcfg.Hq * visible_pairs(L, pcfg.window, pcfg.n_sink, False)
    fa_bytes = float(dcfg.B) * dcfg.Lmax * dcfg.Hkv * dcfg.D * 2 * 2
    swa_bytes = float(dcfg.B) * (dcfg.window + dcfg.n_sink) * dcfg.Hkv * dcfg.D * 2 * 2
    stream = torch.cuda.current_stream()

    def step(events=None):
        full_p = swaa.schedule_is_full(pol_fa_decode, layer, 0)
        full_d = swaa.schedule_is_full(pol_fa_decode, layer, 1)
        full_s = swaa.schedule_is_full(pol_swa_decode, layer, 1)
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(6)] if events is not None else None
        flush_l2()
        if ev: ev[0].record(stream)
        swaa.swaa_prefill(q, k, v, out, cu, L, pcfg.window, pcfg.n_sink, full_p)
        if ev: ev[1].record(stream)
        flush_l2()
        if ev: ev[2].record(stream)
        swaa.swaa_decode(dq, kc, vc, dout, sl, dcfg.window, dcfg.n_sink, full_d, ws_fa)
        if ev: ev[3].record(stream)
        flush_l2()
        if ev: ev[4].record(stream)
        swaa.swaa_decode(dq, kc, vc, dout, sl, dcfg.window, dcfg.n_sink, full_s, ws_swa)
        if ev: ev[5].record(stream)
        if events is not None:
            events.append(ev)
        return full_p, full_d, full_s

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        flags = step()
    assert flags == (False, True, False)
    barrier()
    assert swaa.last_device_status() == 0

    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    launches0 = swaa.kernel_launch_count()
    events = []
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    sampler.start()
    t_start.record(stream)
    for _ in range(args.steps):
        step(events)
    t_end.record(stream)
    barrier()
    clocks = sampler.stop()
    launches = swaa.kernel_launch_count() - launches0
    assert swaa.last_device_status() == 0
    total_ms = t_start.elapsed_time(t_end)
    pre_ms = [e[0].elapsed_time(e[1]) for e in events]
    fa_ms = [e[2].elapsed_time(e[3]) for e in events]
    swa_ms = [e[4].elapsed_time(e[5]) for e in events]
    # per kernel: the median over the timed steps is the reported time (a single slow launch, e.g. one that met a
    # clock change, does not move it); minimum and mean go into the line beside it
    st_pre, st_fa, st_swa = stats_ms(pre_ms), stats_ms(fa_ms), stats_ms(swa_ms)
    t_pre, t_fa, t_swa = st_pre["median"], st_fa["median"], st_swa["median"]

    # ---------------------------------------------------------------- end to end from host buffers
    qh, kh, vh = (t.cpu().pin_memory() for t in (q, k, v))
    outh = torch.empty(out.shape, dtype=out.dtype).pin_memory()
    dqh, douth = dq.cpu().pin_memory(), torch.empty(dout.shape, dtype=dout.dtype).pin_memory()
    q2, k2, v2, dq2 = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v), torch.empty_like(dq)
    e2e_steps = max(3, min(args.steps, 10))

    def e2e_step():
        q2.copy_(qh, non_blocking=True)
        k2.copy_(kh, non_blocking=True)
        v2.copy_(vh, non_blocking=True)
        swaa.swaa_prefill(q2, k2, v2, out, cu, L, pcfg.window, pcfg.n_sink, False)
        outh.copy_(out, non_blocking=True)

    def e2e_decode_step(full, ws):
        dq2.copy_(dqh, non_blocking=True)
        swaa.swaa_decode(dq2, kc, vc, dout, sl, dcfg.window, dcfg.n_sink, full, ws)
        douth.copy_(dout, non_blocking=True)

    def time_loop(fn, n):
        fn()
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n):
            fn()
        b.record(stream)
        barrier()
        return a.elapsed_time(b) / n

    e2e_ms = time_loop(e2e_step, e2e_steps)

    # The same steps pipelined over three streams with two sets of device buffers: the upload of step i + 1 and the
    # download of step i - 1 run beside the kernel of step i (PCIe carries both directions at once).  Every step
    # still uploads its own inputs and downloads its own result; only the waiting is overlapped.
    def e2e_pipelined(n):
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        bufs = [(q2, k2, v2, out), (torch.empty_like(q), torch.empty_like(k), torch.empty_like(v), torch.empty_like(out))]
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_k = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]
        barrier()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        s_in.wait_event(a)
        s_out.wait_event(a)
        for i in range(n):
            qd, kd, vd, od = bufs[i % 2]
            with torch.cuda.stream(s_in):
                if i >= 2:
                    s_in.wait_event(ev_k[i % 2])      # the kernel of step i - 2 has read these inputs
                qd.copy_(qh, non_blocking=True)
                kd.copy_(kh, non_blocking=True)
                vd.copy_(vh, non_blocking=True)
                ev_in[i % 2].record(s_in)
            stream.wait_event(ev_in[i % 2])
            if i >= 2:
                stream.wait_event(ev_out[i % 2])      # the download of step i - 2 has read this output
            swaa.swaa_prefill(qd, kd, vd, od, cu, L, pcfg.window, pcfg.n_sink, False)
            ev_k[i % 2].record(stream)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_k[i % 2])
                outh.copy_(od, non_blocking=True)
                ev_out[i % 2].record(s_out)
        stream.wait_event(ev_out[(n - 1) % 2])
        if n >= 2:
            stream.wait_event(ev_out[(n - 2) % 2])
        b.record(stream)
        barrier()
        del bufs
        return a.elapsed_time(b) / n

    e2e_pipe_ms = e2e_pipelined(max(6, e2e_steps))
    e2e_fa_ms = time_loop(lambda: e2e_decode_step(True, ws_fa), e2e_steps)
    e2e_swa_ms = time_loop(lambda: e2e_decode_step(False, ws_swa), e2e_steps)

    # ---------------------------------------------------------------- max over ranks
    total_ms, t_pre, t_fa, t_swa, e2e_ms, e2e_fa_ms, e2e_swa_ms, e2e_pipe_ms = max_over_ranks(
        [total_ms, t_pre, t_fa, t_swa, e2e_ms, e2e_fa_ms, e2e_swa_ms, e2e_pipe_ms], world, dev)
    K, N = args.steps, world


    # ---------------------------------------------------------------- backward pass of the same layer (outside the timed step)
    backward = None
    if rank == 0 and N == 1:
        T, Hq, D = q.shape
        lse = torch.empty((Hq, T), dtype=torch.float32, device=dev)
        swaa.swaa_prefill(q, k, v, out, cu, L, pcfg.window, pcfg.n_sink, False, lse=lse)
        grad_out = torch.randn(q.shape, device=dev).to(torch.bfloat16)
        dq_, dk_, dv_ = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        bws = torch.empty(swaa.prefill_backward_workspace_size(1, T, Hq, pcfg.Hkv, D, pcfg.n_sink), dtype=torch.uint8, device=dev)
        bms = []
        for r in range(6):
            flush_l2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            swaa.swaa_prefill_backward(q, k, v, out, grad_out, lse, cu, L, pcfg.window, pcfg.n_sink, False, dq_, dk_, dv_, bws)
            b.record(stream)
            torch.cuda.synchronize()
            if r > 0:
                bms.append(a.elapsed_time(b))
        if swaa.last_device_status() != 0:
            raise RuntimeError("swaa_prefill_backward reported a device error")
        bms.sort()
        btf = 2.5 * prefill_flops / (bms[len(bms) // 2] * 1e-3) / 1e12  # five products where the forward pass has two
        backward = {"ms": bms[len(bms) // 2], "effective_tflops": btf, "frac_of_measured_peak": btf / peaks["bf16_tflops"],
                    "note": "swaa_prefill_backward on the same workload, whole call, median of 5, L2 flushed; not part of the step"}
        del lse, grad_out, dq_, dk_, dv_, bws

    # ---------------------------------------------------------------- the other workloads and the L sweep (N = 1)
    extra = None
    if rank == 0 and N == 1 and not args.no_extra:
        extra = run_extra_workloads(swaa, torch, inputs, flush_l2, stream, peaks)

    cpu_baseline = None
    if rank == 0 and N == 1:
        import oracle

        qf, kf, vf = (inputs.to_f32_numpy(t) for t in (q, k, v))
        rng = np.random.default_rng(1234)

        def oracle_rows(n):
            rt = rng.integers(pcfg.window + pcfg.n_sink, L, n)
            rh = rng.integers(0, pcfg.Hq, n).astype(np.int32)
            t0 = time.perf_counter()
            r = oracle.prefill(qf, kf, vf, [0, L], pcfg.window, pcfg.n_sink, False, rows=(rt, rh))
            return time.perf_counter() - t0, 4.0 * pcfg.D * float(r["nvis"].sum())

        dt, _ = oracle_rows(512)
        n_rows = int(max(512, min(1 << 20, 512 * 15.0 / max(dt, 1e-6))))  # about 15 s of CPU work
        dt, fl = oracle_rows(n_rows)
        cpu_baseline = {"value": fl / dt / 1e12, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                        "sample": f"{n_rows} seeded (row, head) rows of the same workload, {dt:.1f} s"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return
    avg_pre_ms = t_pre  # median over the timed steps (max over ranks)
    achieved = whole_job_value(prefill_flops, 1, avg_pre_ms * 1e-3) / 1e12  # per GPU; the line reports N x this
    fa_gbs = fa_bytes / (t_fa * 1e-3) / 1e9
    swa_gbs = swa_bytes / (t_swa * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": N * achieved, "unit": UNIT, "n_gpus": N, "steps": K, "warmup": max(args.warmup, 3),
        "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": "cfg2 long-context SWA prefill: B=1 L=32768 Hq=32 Hkv=8 D=128 W=2048 n_sink=4 "
                               "(K row 0 shifted); step also runs cfg4 decode B=16 Lcache=65536 FA and SWA(W=4096,n_sink=4)",
                   "l2": "flushed before every kernel: 256 MiB write, then 256 MiB read (clean lines)", "parallelism": f"replicas x{N}",
                   "value_from": "median over the timed steps of the prefill kernel time inside the step "
                                 "(CUDA events on the launching stream)"},
        "clocks": clocks,
        "e2e": {"value": N * prefill_flops / (e2e_pipe_ms * 1e-3) / 1e12, "unit": UNIT,
                "h2d_bytes_per_step": int(q.numel() + k.numel() + v.numel()) * 2, "d2h_bytes_per_step": int(out.numel()) * 2,
                "ms_per_step": e2e_pipe_ms,
                "how": "every step uploads its Q, K, V from pinned host memory, runs swaa_prefill and downloads `out`; "
                       "upload, kernel and download of neighbouring steps overlap (three streams, two device buffer sets)",
                "serial": {"value": N * prefill_flops / (e2e_ms * 1e-3) / 1e12, "ms_per_step": e2e_ms,
                           "how": "the same on one stream, nothing overlapped"}},
        "gpu_launches": int(launches),
        "roofline": {"kernel": "prefill_kernel<128, 0>", "bound": "tensor", "achieved": achieved,
                     "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"],
                     "traffic": PREFILL_DRAM_TRAFFIC_BYTES, "peak_source": peaks["source"] + " burst bf16",
                     "frac_of_nominal_2250": achieved / 2250.0, "ms_per_launch": avg_pre_ms,
                     "ms_per_launch_min": st_pre["min"], "ms_per_launch_mean": st_pre["mean"],
                     "achieved_at_min": prefill_flops / (st_pre["min"] * 1e-3) / 1e12},
        "decode": {
            "fa": {"gbs": N * fa_gbs, "us_per_launch": 1e3 * t_fa, "us_per_launch_min": 1e3 * st_fa["min"],
                   "us_per_launch_mean": 1e3 * st_fa["mean"], "bytes": fa_bytes,
                   "roofline": {"bound": "hbm", "achieved": fa_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                "frac": fa_gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": fa_gbs / 8000.0,
                                "traffic": DECODE_FA_DRAM_TRAFFIC_BYTES},
                   "e2e_gbs": fa_bytes / (e2e_fa_ms * 1e-3) / 1e9},
            "swa": {"gbs": N * swa_gbs, "us_per_launch": 1e3 * t_swa, "us_per_launch_min": 1e3 * st_swa["min"],
                    "us_per_launch_mean": 1e3 * st_swa["mean"], "bytes": swa_bytes,
                    "roofline": {"bound": "hbm", "achieved": swa_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                 "frac": swa_gbs / peaks["hbm_gbs"], "frac_of_nominal_8000": swa_gbs / 8000.0,
                                 "traffic": DECODE_SWA_DRAM_TRAFFIC_BYTES},
                    "e2e_gbs": swa_bytes / (e2e_swa_ms * 1e-3) / 1e9},
        },
        "backward": backward,
        "extra": extra,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_extra_workloads(swaa, torch, inputs, flush_l2, stream, peaks):
    """The workloads the timed step does not contain, one flushed launch set each, after the timed steps: workload
    1 (tiny), workload 5 (varlen), the time against L at fixed W (App. A: O(N * W)), and workload 3, the 36-layer
    interleaved stack with its mask policy from the layer schedule (per kind and in total; the stack runs for
    seconds, so its total is set against the sustained bf16 peak)."""
    extra = {"note": "outside the timed step; median of `launches` launches each, L2 flushed before every launch; the GPU "
                     "idles for half a second before each case so that the power state of the case before it (the "
                     "backward pass, the varlen batch) does not carry over; light cases first"}

    def settled(*a, **kw):
        torch.cuda.synchronize()
        time.sleep(0.5)
        return time_prefill_case(swaa, torch, flush_l2, stream, peaks, *a, **kw)

    extra["cfg1_tiny"] = settled(inputs.cfg_tiny(), False, 5)
    extra["linear_in_L"] = [settled(inputs.cfg_long(L=L), False, 5) for L in (8192, 16384, 32768, 65536, 131072)]
    extra["cfg5_varlen"] = settled(inputs.cfg_varlen(), False, 3)
    torch.cuda.synchronize()
    time.sleep(0.5)
    pol = swaa.SwaaPolicy(n_layers=36, window=4096, n_sink=64, fa_start=3, fa_step=4, fa_decode=True)
    per_kind, flops = {False: [], True: []}, 0.0
    tensors = None
    for layer in range(pol.n_layers):
        cfg = inputs.cfg_stack_layer(layer)
        full = swaa.schedule_is_full(pol, layer, 0)
        del tensors
        tensors = inputs.make_prefill_inputs(cfg, "cuda")
        r = time_prefill_case(swaa, torch, flush_l2, stream, peaks, cfg, full, 1, tensors=tensors)
        per_kind[bool(full)].append(r["ms"])
        flops += r["effective_tflops"] * r["ms"] * 1e9
    del tensors
    total = sum(per_kind[False]) + sum(per_kind[True])
    tf = flops / (total * 1e-3) / 1e12
    extra["cfg3_stack"] = {
        "layers": pol.n_layers, "ms_total": total, "effective_tflops": tf,
        "frac_of_measured_sustained_peak": tf / peaks["bf16_tflops_sustained"], "frac_of_nominal_2250": tf / 2250.0,
        "swa_layers": len(per_kind[False]), "ms_per_swa_layer": sum(per_kind[False]) / len(per_kind[False]),
        "ms_swa_layer_min": min(per_kind[False]), "ms_swa_layer_max": max(per_kind[False]),
        "fa_layers": len(per_kind[True]), "ms_per_fa_layer": sum(per_kind[True]) / len(per_kind[True]),
        "launches_per_layer": 1}
    return extra


def run_profile_case(case: str):
    """A few launches of one kernel on its benchmark workload and nothing else: the command that the
    ncu captures summarised under profiles/ run."""
    import torch

    import paper_2512_10411_b200 as swaa
    from paper_2512_10411_b200 import inputs

    torch.cuda.set_device(0)
    if case.startswith("prefill"):
        cfg = {"prefill": inputs.cfg_long(), "prefill_full": inputs.cfg_long(is_full=True),
               "prefill_tiny": inputs.cfg_tiny()}[case]
        q, k, v, cu = inputs.make_prefill_inputs(cfg, "cuda")
        out = torch.empty_like(q)
        for _ in range(3):
            swaa.swaa_prefill(q, k, v, out, cu, cfg.seqlens[0], cfg.window, cfg.n_sink, cfg.is_full)
    elif case == "backward":
        # heads and mask of workload 2 at a quarter of its length (0.5 GB on the device with the fp32 workspace)
        cfg = inputs.PrefillConfig("backward_L8192", (8192,), 32, 8, 128, 2048, 4, False, seed=2)
        q, k, v, cu = inputs.make_prefill_inputs(cfg, "cuda")
        T, Hq, D = q.shape
        out, dout = torch.empty_like(q), torch.randn(q.shape, device="cuda").to(torch.bfloat16)
        lse = torch.empty((Hq, T), dtype=torch.float32, device="cuda")
        swaa.swaa_prefill(q, k, v, out, cu, cfg.seqlens[0], cfg.window, cfg.n_sink, False, lse=lse)
        dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
        ws = torch.empty(swaa.prefill_backward_workspace_size(1, T, Hq, cfg.Hkv, D, cfg.n_sink), dtype=torch.uint8,
                         device="cuda")
        for _ in range(3):
            swaa.swaa_prefill_backward(q, k, v, out, dout, lse, cu, cfg.seqlens[0], cfg.window, cfg.n_sink, False, dq, dk,
                                       dv, ws)
    else:
        cfg = inputs.cfg_decode(B=4) if case.endswith("_small") else inputs.cfg_decode()
        full = "fa" in case
        q, kc, vc, sl = inputs.make_decode_inputs(cfg, "cuda")
        ws = torch.empty(swaa.decode_workspace_size(cfg.B, cfg.Hq, cfg.Hkv, cfg.D, cfg.Lmax, cfg.window, cfg.n_sink,
                                                    full), dtype=torch.uint8, device="cuda")
        out = torch.empty_like(q)
        for _ in range(3):
            swaa.swaa_decode(q, kc, vc, out, sl, cfg.window, cfg.n_sink, full, ws)
    assert swaa.last_device_status() == 0
    print(json.dumps({"profile_case": case, "launches": swaa.kernel_launch_count()}))


def run_sweep():
    """Times swaa_prefill on the other workloads and on the parameter sweeps that show how the time depends
    on L, W and n_sink (one GPU; median of a few launches, L2 flushed before each; one JSON line per case)."""
    import dataclasses

    import torch

    import paper_2512_10411_b200 as swaa
    from paper_2512_10411_b200 import inputs

    torch.cuda.set_device(0)
    peaks = load_peaks()
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device="cuda")
    flush_rd = torch.zeros(L2_FLUSH_BYTES // 4, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def flush_l2():
        flush.zero_()
        flush_rd.sum()

    def time_case(tag, cfg, is_full, reps=5, tensors=None):
        line = {"case": tag}
        line.update(time_prefill_case(swaa, torch, flush_l2, stream, peaks, cfg, is_full, reps, tensors=tensors))
        print(json.dumps(line), flush=True)
        return line["ms"]

    # time against L at fixed W (App. A: O(N*W)), then the sink and window variants on workload 2
    for L in (8192, 16384, 32768, 65536, 131072):
        time_case("linear_in_L", inputs.cfg_long(L=L), False)
    for S in (0, 4, 100):
        time_case("sinks", inputs.cfg_long(n_sink=S), False)
    for W in (1024, 2048, 4096, 8192):
        time_case("window", inputs.cfg_long(window=W), False)
    time_case("cfg2_full_causal", inputs.cfg_long(is_full=True), True, reps=3)
    time_case("cfg5_varlen", inputs.cfg_varlen(), False, reps=3)
    time_case("cfg1_tiny", inputs.cfg_tiny(), False)
    # backward pass on workload 2 (five tile products per visible pair: 10 * D * Hq * pairs FLOP)
    bcfg = inputs.cfg_long()
    bq, bk, bv, bcu = inputs.make_prefill_inputs(bcfg, "cuda")
    bT, bHq, bD = bq.shape
    bout, bdo = torch.empty_like(bq), torch.randn(bq.shape, device="cuda").to(torch.bfloat16)
    blse = torch.empty((bHq, bT), dtype=torch.float32, device="cuda")
    swaa.swaa_prefill(bq, bk, bv, bout, bcu, bcfg.seqlens[0], bcfg.window, bcfg.n_sink, False, lse=blse)
    bdq, bdk, bdv = torch.empty_like(bq), torch.empty_like(bk), torch.empty_like(bv)
    bws = torch.empty(swaa.prefill_backward_workspace_size(1, bT, bHq, bcfg.Hkv, bD, bcfg.n_sink), dtype=torch.uint8, device="cuda")
    ms = []
    for r in range(4):
        flush.zero_()
        flush_rd.sum()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        swaa.swaa_prefill_backward(bq, bk, bv, bout, bdo, blse, bcu, bcfg.seqlens[0], bcfg.window, bcfg.n_sink, False, bdq,
                                   bdk, bdv, bws)
        b.record(stream)
        torch.cuda.synchronize()
        if r > 0:
            ms.append(a.elapsed_time(b))
    assert swaa.last_device_status() == 0
    ms.sort()
    bflops = 10.0 * bD * bHq * visible_pairs(bcfg.seqlens[0], bcfg.window, bcfg.n_sink, False)
    tf = bflops / (ms[len(ms) // 2] * 1e-3) / 1e12
    print(json.dumps({"case": "backward_cfg2", "L": bcfg.seqlens[0], "Hq": bHq, "Hkv": bcfg.Hkv, "D": bD,
                      "window": bcfg.window, "n_sink": bcfg.n_sink, "ms": ms[len(ms) // 2], "effective_tflops": tf,
                      "frac_of_measured_peak": tf / peaks["bf16_tflops"]}), flush=True)
    del bq, bk, bv, bout, bdo, bdq, bdk, bdv, bws
    # chunked prefill: a 4096-token chunk at the end of a 131072-token context (heads and mask of workload 2)
    g = torch.Generator(device="cuda").manual_seed(7)
    lq, lk, Hq, Hkv, D, W, S = 4096, 131072, 32, 8, 128, 2048, 4
    cq = torch.randn((lq, Hq, D), generator=g, device="cuda").to(torch.bfloat16)
    ck = torch.randn((lk, Hkv, D), generator=g, device="cuda").to(torch.bfloat16)
    cv = torch.randn((lk, Hkv, D), generator=g, device="cuda").to(torch.bfloat16)
    cuq = torch.tensor([0, lq], dtype=torch.int32, device="cuda")
    cuk = torch.tensor([0, lk], dtype=torch.int32, device="cuda")
    cout = torch.empty_like(cq)
    for full in (False, True):
        ms = []
        for r in range(6):
            flush.zero_()
            flush_rd.sum()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            swaa.swaa_prefill_chunked(cq, ck, cv, cout, cuq, cuk, lq, lk, W, S, full)
            b.record(stream)
            torch.cuda.synchronize()
            if r > 0:
                ms.append(a.elapsed_time(b))
        assert swaa.last_device_status() == 0
        ms.sort()
        pairs = sum(lk - lq + i + 1 for i in range(lq)) if full else lq * (W + S)
        tf = 4.0 * D * Hq * pairs / (ms[len(ms) // 2] * 1e-3) / 1e12
        print(json.dumps({"case": "chunked_prefill", "len_q": lq, "len_k": lk, "Hq": Hq, "Hkv": Hkv, "D": D, "window": W,
                          "n_sink": S, "is_full": full, "ms": ms[len(ms) // 2], "effective_tflops": tf,
                          "frac_of_measured_peak": tf / peaks["bf16_tflops"]}), flush=True)
    # the same chunk against a paged pool (256-entry pages in random order)
    pg = 256
    nb = lk // pg
    perm = torch.randperm(nb, generator=g, device="cuda")
    pkp = torch.empty((nb, pg, Hkv, D), dtype=torch.bfloat16, device="cuda")
    pvp = torch.empty_like(pkp)
    pkp[perm] = ck.view(nb, pg, Hkv, D)
    pvp[perm] = cv.view(nb, pg, Hkv, D)
    pbt = perm.view(1, nb).to(torch.int32).contiguous()
    psk = torch.tensor([lk], dtype=torch.int32, device="cuda")
    ms = []
    for r in range(6):
        flush.zero_()
        flush_rd.sum()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        swaa.swaa_prefill_paged(cq, pkp, pvp, cout, cuq, psk, pbt, lq, W, S, False)
        b.record(stream)
        torch.cuda.synchronize()
        if r > 0:
            ms.append(a.elapsed_time(b))
    assert swaa.last_device_status() == 0
    ms.sort()
    tf = 4.0 * D * Hq * lq * (W + S) / (ms[len(ms) // 2] * 1e-3) / 1e12
    print(json.dumps({"case": "paged_chunked_prefill", "len_q": lq, "len_k": lk, "page_size": pg, "window": W, "n_sink": S,
                      "is_full": False, "ms": ms[len(ms) // 2], "effective_tflops": tf,
                      "frac_of_measured_peak": tf / peaks["bf16_tflops"]}), flush=True)
    del cq, ck, cv, cout, pkp, pvp
    # paged decode: workload 4 with 256-entry pages handed out in random order, against the dense layout
    dcfg = inputs.cfg_decode()
    dq, kc, vc, sl = inputs.make_decode_inputs(dcfg, "cuda")
    page = 256
    nblk = dcfg.Lmax // page
    perm = torch.randperm(dcfg.B * nblk, generator=g, device="cuda")
    bt = perm.view(dcfg.B, nblk).to(torch.int32).contiguous()
    kp = torch.empty((dcfg.B * nblk, page, dcfg.Hkv, dcfg.D), dtype=torch.bfloat16, device="cuda")
    vp = torch.empty_like(kp)
    kp[perm] = kc.view(dcfg.B * nblk, page, dcfg.Hkv, dcfg.D)
    vp[perm] = vc.view(dcfg.B * nblk, page, dcfg.Hkv, dcfg.D)
    dout = torch.empty_like(dq)
    for full in (True, False):
        nbytes = float(dcfg.B) * (dcfg.Lmax if full else dcfg.window + dcfg.n_sink) * dcfg.Hkv * dcfg.D * 4
        ws_d = torch.empty(swaa.decode_workspace_size(dcfg.B, dcfg.Hq, dcfg.Hkv, dcfg.D, dcfg.Lmax, dcfg.window,
                                                      dcfg.n_sink, full), dtype=torch.uint8, device="cuda")
        ws_p = torch.empty(swaa.decode_paged_workspace_size(dcfg.B, dcfg.Hq, dcfg.Hkv, dcfg.D, nblk, page, dcfg.window,
                                                            dcfg.n_sink, full), dtype=torch.uint8, device="cuda")
        res = {}
        for kind in ("dense", "paged"):
            us = []
            for r in range(11):
                flush.zero_()
                flush_rd.sum()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                if kind == "dense":
                    swaa.swaa_decode(dq, kc, vc, dout, sl, dcfg.window, dcfg.n_sink, full, ws_d)
                else:
                    swaa.swaa_decode_paged(dq, kp, vp, dout, bt, sl, dcfg.window, dcfg.n_sink, full, ws_p)
                b.record(stream)
                torch.cuda.synchronize()
                if r > 0:
                    us.append(1e3 * a.elapsed_time(b))
            us.sort()
            res[kind] = us[len(us) // 2]
        assert swaa.last_device_status() == 0
        print(json.dumps({"case": "decode_paged_vs_dense", "is_full": full, "page_size": page, "bytes": nbytes,
                          "dense_us": res["dense"], "dense_gbs": nbytes / res["dense"] / 1e3,
                          "paged_us": res["paged"], "paged_gbs": nbytes / res["paged"] / 1e3,
                          "hbm_peak_gbs": peaks["hbm_gbs"]}), flush=True)
    del kc, vc, kp, vp
    # workload 3: the 36-layer interleaved stack, per layer and in total (mask policy from the layer schedule)
    pol = swaa.SwaaPolicy(n_layers=36, window=4096, n_sink=64, fa_start=3, fa_step=4, fa_decode=True)
    total, per_kind = 0.0, {False: [], True: []}
    for layer in range(pol.n_layers):
        cfg = inputs.cfg_stack_layer(layer)
        full = swaa.schedule_is_full(pol, layer, 0)
        t = time_case(f"cfg3_layer{layer:02d}", cfg, full, reps=1)
        total += t
        per_kind[bool(full)].append(t)
    print(json.dumps({"case": "cfg3_stack_total", "layers": pol.n_layers, "ms_total": total,
                      "swa_layers": len(per_kind[False]), "ms_per_swa_layer": sum(per_kind[False]) / len(per_kind[False]),
                      "fa_layers": len(per_kind[True]), "ms_per_fa_layer": sum(per_kind[True]) / len(per_kind[True])}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--profile-case", default=None,
                    choices=["prefill", "prefill_full", "prefill_tiny", "backward", "decode_fa", "decode_swa",
                             "decode_fa_small", "decode_swa_small"],
                    help="run three launches of one kernel only (for ncu) and exit")
    ap.add_argument("--no-extra", action="store_true",
                    help="skip the workloads outside the timed step (workloads 1, 3, 5 and the L sweep)")
    ap.add_argument("--decode-split", action="store_true",
                    help="decode workload 4 with the cache cut along the context over the ranks (or, on one GPU, over "
                         "--shards shards run in sequence) and exit")
    ap.add_argument("--shards", type=int, default=4)
    ap.add_argument("--context-parallel", action="store_true",
                    help="SWA prefill of workload 2 cut along the context over the ranks (halo + sink exchange, then "
                         "swaa_prefill_context_parallel) and exit")
    ap.add_argument("--sweep", action="store_true",
                    help="time swaa_prefill on the other workloads and the L / W / n_sink sweeps (one GPU) and exit")
    args = ap.parse_args()
    if args.sweep:
        run_sweep()
        return
    if args.profile_case:
        run_profile_case(args.profile_case)
        return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.context_parallel:
        run_context_parallel(args, rank, local_rank, world)
    elif args.decode_split:
        run_decode_split(args, rank, local_rank, world)
    elif args.impl == "reference":
        run_reference(args, rank)
    else:
        run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()

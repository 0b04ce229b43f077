#!/usr/bin/env python
"""Benchmark of the encoder forward (metric: sequences/s and p50 latency of one forward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c2] [--impl ours|reference]

One "step" is one forward of the whole hot path (embedding+LN, L encoder layers, pool+L2) over one
batch of seeded synthetic inputs.  Default workload: the headline configuration (MiniLM-L6 shape,
batch 32, seq 128).  With N > 1 (launched by torchrun, one rank per GPU) every rank runs the same
workload on its own batch (weak scaling, no data-path collective); times are the max over ranks.

Prints ONE JSON line.  `value` is device-timed throughput with inputs resident in HBM; `e2e` is the
same metric through the host-buffer C-ABI call (H2D copy of ids/mask, forward, D2H copy of the
embeddings, stream sync inside the timed region); `roofline` describes the dominant kernel;
`cpu_baseline` is the fp64 oracle on host cores.  With the default workload (c2) the same line also
carries `roofline_c3`: the per-kernel table of the roofline configuration (batch 256 x seq 256).
`--impl reference` times the oracle itself (a deliberately slow, plain program).

Per-kernel times.  The forward is replayed as one CUDA graph with programmatic dependent launch between
its kernels; that replay, untouched, gives the step time.  A second encoder replays the same graph with
event-record nodes between the kernels: those intervals serialise the kernels and carry a few
microseconds of event overhead each, so they are used only to SPLIT the untouched step time among the
kernels, in proportion to the intervals (the kernels' shares are the intervals' shares, the same
shares a serialised profiler launch list shows; the kernels' times add up to the step time).
`achieved` = algorithmic work / that time; the raw interval is reported next to it.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "encoder forward sequences/s (p50 ms reported alongside)"
KERNEL_CLASSES = ("gemm_qkv", "attention", "gemm_out", "ln1", "gemm_ffn1", "gemm_ffn2", "ln2")


def load_dram_traffic():
    """dram__bytes per launch from the ncu captures, read from the table in profiles/dram_traffic.md
    (rows: | workload | kernel class | MB per launch | summary file |).  Missing file or row -> None."""
    table = {}
    path = os.path.join(ROOT, "profiles", "dram_traffic.md")
    try:
        with open(path) as f:
            for line in f:
                cells = [c.strip() for c in line.strip().strip("|").split("|")]
                if len(cells) >= 3 and cells[0] in ("c0", "c1", "c2", "c3", "c4"):
                    try:
                        table.setdefault(cells[0], {})[cells[1]] = float(cells[2])
                    except ValueError:
                        pass
    except OSError:
        pass
    return table

# B200: 148 SMs x 16 special-function results per clock x 1.965 GHz (exp2 of the softmax)
EXP_PEAK_TEXP_S = 148 * 16 * 1.965e9 / 1e12
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return p, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


def usable_cores() -> int:
    try:
        return len(os.sched_getaffinity(0))
    except Exception:
        return os.cpu_count() or 1


# ---------------------------------------------------------------------------- clocks
class ClockSampler(threading.Thread):
    """Polls SM clock and throttle reasons through NVML (read-only) while the timed region runs."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, torch_device_index: int):
        super().__init__(daemon=True)
        self.samples, self.reason_bits, self.max_mhz = [], 0, None
        self._stop_evt = threading.Event()
        self.active = threading.Event()
        self.handle = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            uuid = str(torch.cuda.get_device_properties(torch_device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            try:
                self.handle = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(torch_device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.handle, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.handle = None

    def run(self):
        if self.handle is None:
            return
        while not self._stop_evt.is_set():
            if self.active.is_set():
                try:
                    self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.handle, self.nv.NVML_CLOCK_SM))
                    self.reason_bits |= int(self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle))
                except Exception:
                    pass
            time.sleep(0.005)

    def stop(self):
        self._stop_evt.set()

    def summary(self):
        reasons = [n for bit, n in self.REASONS.items() if self.reason_bits & bit and n != "gpu_idle"]
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": reasons, "samples": len(self.samples)}


# ---------------------------------------------------------------------------- oracle timing
def time_oracle(cfg_name: str, budget_s: float, steps: int = 1, warmup: int = 0, all_valid: bool = False):
    """Times the fp64 oracle (as it stands) on host cores on a bounded sample of the workload:
    the first n sequences of the seeded batch, n chosen from a one-sequence calibration run so
    that one step costs about `budget_s` seconds."""
    from oracle import oracle
    from synth.inputs import CONFIGS, EncoderConfig, make_inputs

    cfg = CONFIGS[cfg_name]
    inp = make_inputs(cfg, lengths=np.full(cfg.batch, cfg.seq, dtype=np.int64) if all_valid else None)
    cores = usable_cores()
    oracle.set_threads(cores)

    last_out = {}

    def run(n):
        sub = EncoderConfig(**{**cfg.__dict__, "batch": n})
        t0 = time.perf_counter()
        last_out["emb"] = oracle.encoder_forward(sub, inp.ids[:n], inp.mask[:n], inp.params, inp.layers)
        return time.perf_counter() - t0

    run(1)  # builds/loads the library, warms caches
    t1 = run(1)
    n = int(max(1, min(cfg.batch, budget_s / max(t1, 1e-6))))
    for _ in range(warmup):
        run(n)
    times = [run(n) for _ in range(max(steps, 1))]
    return {"times": times, "n": n, "cores": cores, "batch": cfg.batch, "embeddings": last_out["emb"]}


def run_reference_arm(args):
    """--impl reference: the oracle is the reference arm of this build (no upstream code exists)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    total_budget = 150.0
    per_step = total_budget / max(args.steps + args.warmup, 1)
    r = time_oracle(args.config, per_step, steps=args.steps, warmup=args.warmup, all_valid=args.all_valid)
    mean_t = sum(r["times"]) / len(r["times"])
    value = r["n"] / mean_t
    sample = f"first {r['n']} of {r['batch']} sequences of {args.config} per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "sequences/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": mean_t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(args.config, extra={"sample": sample}),
        "cpu_baseline": {"value": value, "unit": "sequences/s", "cores": r["cores"], "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "sequences/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def workload_config(name: str, extra=None):
    from synth.inputs import CONFIGS
    c = CONFIGS[name]
    d = {"workload": f"{name}: {c.num_layers}-layer encoder, hidden {c.hidden}, {c.num_heads} heads, ffn {c.ffn}, "
                     f"batch {c.batch} x seq {c.seq}, valid lengths uniform in [{c.len_lo},{c.len_hi}]",
         "batch_per_gpu": c.batch, "seq_len": c.seq, "l2": "flushed between timed iterations (256 MiB write)",
         "parallelism": "replicated weights, batch sharded across ranks, no collective"}
    if extra:
        d.update(extra)
        if "valid_lengths" in extra:
            d["workload"] = d["workload"].replace(f"valid lengths uniform in [{c.len_lo},{c.len_hi}]", "every sequence full length")
    return d


# ---------------------------------------------------------------------------- roofline bookkeeping
def kernel_classes(num_layers: int, fused_ln: bool, fused_ffn: bool = False):
    per_layer = [k for k in KERNEL_CLASSES if not (fused_ln and k in ("ln1", "ln2"))]
    if fused_ffn:   # everything behind the attention is one kernel
        per_layer = ["gemm_qkv", "attention", "layer_tail"]
    names = ["pack", "embed_ln"]
    for _ in range(num_layers):
        names += per_layer
    names.append("pool_l2")
    return names


def algorithmic_work(cls: str, c, lengths):
    """(bound, work per launch, unit).  Valid tokens are packed, so only they are computed and only
    they are counted: T = sum of valid lengths rows for the GEMMs and row kernels, sum of len^2
    query-key pairs for attention.  Skipped (padded) work is never counted."""
    H, F, S, B = c.hidden, c.ffn, c.seq, c.batch
    T = int(np.sum(lengths))
    n_valid_tokens = T
    pairs = float(np.sum(np.asarray(lengths, dtype=np.float64) ** 2))
    if cls == "pack":
        return "hbm", B * S * 4.0 + T * 4.0 + B * 8.0, "byte"   # read the mask, write positions and offsets
    if cls == "gemm_qkv":
        return "tensor", 2.0 * T * 3 * H * H, "flop"
    if cls == "gemm_out":
        return "tensor", 2.0 * T * H * H, "flop"
    if cls in ("gemm_ffn1", "gemm_ffn2"):
        return "tensor", 2.0 * T * F * H, "flop"
    if cls == "layer_tail":
        return "tensor", 4.0 * T * F * H + 2.0 * T * H * H, "flop"
    if cls == "attention":
        # at head_dim 32/64 the softmax exponentials (one per query-key pair and head), not the
        # QK^T / PV flops, are the scarce resource: 128..256 flops per exp against a tensor : MUFU
        # throughput ratio of ~3500 : 1
        return "alu", pairs * c.num_heads, "exp"
    if cls in ("ln1", "ln2"):
        return "hbm", 2.0 * T * H * 2, "byte"                 # read + write one bf16 row per token
    if cls == "embed_ln":
        return "hbm", T * (2.0 * H * 2 + 4), "byte"           # word-row gather + output row + id
    if cls == "pool_l2":
        return "hbm", n_valid_tokens * H * 2.0 + B * 8 + B * H * 4, "byte"
    raise KeyError(cls)


# ---------------------------------------------------------------------------- our arm
def gemm_bytes(cls: str, c, T: int):
    """Algorithmic HBM bytes of a projection (activations in and out once, residual once, weights once)."""
    H, F = c.hidden, c.ffn
    if cls == "gemm_qkv":
        return T * (H + 3 * H) * 2.0 + 3 * H * H * 2.0
    if cls == "gemm_out":
        return T * (H + H + H) * 2.0 + H * H * 2.0
    if cls == "gemm_ffn1":
        return T * (H + F) * 2.0 + F * H * 2.0
    if cls == "layer_tail":   # reads ctx and the layer's input rows, writes its output rows; three weight matrices
        return T * (H + H + H) * 2.0 + (2.0 * F * H + H * H) * 2.0
    return T * (F + H + H) * 2.0 + F * H * 2.0   # gemm_ffn2


def kernel_table(cfg, lengths, names, per_class_raw, step_ms, peaks):
    """Splits the untouched step time among the kernel classes (see the module docstring) and sets
    every class against its roofline."""
    n_kernels = len(names)
    raw = {cls: sum(v) / len(v) for cls, v in per_class_raw.items()}                 # ms per launch, event nodes
    tot_raw = sum(raw[cls] * names.count(cls) for cls in raw)
    overhead = max(0.0, (tot_raw - step_ms) / n_kernels)                             # ms per launch, reported only
    scale = step_ms / tot_raw if tot_raw > 0 else 1.0                                # shares = the intervals' shares
    T = int(np.sum(lengths))
    ktab = {}
    for cls in raw:
        t_ms = raw[cls] * scale
        launches = names.count(cls)
        bound, work, unit = algorithmic_work(cls, cfg, lengths)
        row = {"avg_us": t_ms * 1e3, "event_interval_us": raw[cls] * 1e3, "launches_per_step": launches,
               "ms_per_step": t_ms * launches, "share": t_ms * launches / step_ms, "bound": bound}
        if bound == "tensor":
            ach, peak, u = work / (t_ms * 1e-3) / 1e12, peaks["bf16_tflops"], "TFLOP/s"
            # a projection's own floor: the slower of its tensor time and its HBM time
            hbm_us = gemm_bytes(cls, cfg, T) / (peaks["hbm_gbs"] * 1e9) * 1e6
            tensor_us = work / (peak * 1e12) * 1e6
            row.update({"floor_us": max(hbm_us, tensor_us), "floor": "hbm" if hbm_us > tensor_us else "tensor",
                        "frac_of_floor": max(hbm_us, tensor_us) / (t_ms * 1e3)})
        elif bound == "alu":
            ach, peak, u = work / (t_ms * 1e-3) / 1e12, EXP_PEAK_TEXP_S, "Texp/s"
        else:
            ach, peak, u = work / (t_ms * 1e-3) / 1e9, peaks["hbm_gbs"], "GB/s"
        row.update({"achieved": ach, "unit": u, "peak": peak, "frac": ach / peak})
        ktab[cls] = row
    return ktab, overhead * 1e3


class EncoderRun:
    """One workload on this rank: buffers, two encoders (plain / with event nodes), timed regions."""

    def __init__(self, cfg_name, args, rank, local):
        import torch
        import paper_2609_37916_b200 as rlx
        from paper_2609_37916_b200 import binding
        from synth.inputs import CONFIGS, EncoderConfig, make_inputs
        self.torch, self.cfg = torch, CONFIGS[cfg_name]
        cfg = self.cfg
        # --all-valid: every sequence fills the whole padded length (mask all ones), for like-for-like context
        # with benchmarks that feed unpadded inputs; the seeded draw order of everything else is unchanged
        full = np.full(cfg.batch, cfg.seq, dtype=np.int64) if args.all_valid else None
        self.base = make_inputs(cfg, lengths=full)
        if rank == 0:
            self.mine = self.base
        else:  # every rank gets its own batch (ids, lengths) and the same replicated weights
            self.mine = make_inputs(EncoderConfig(**{**cfg.__dict__, "seed": cfg.seed + 1000 * rank}), weights=False, lengths=full)
        self.weights = rlx.upload_weights(self.base.params, self.base.layers)
        B, S, H = cfg.batch, cfg.seq, cfg.hidden
        self.stream = torch.cuda.Stream()
        self.enc = rlx.Encoder.from_config(cfg, max_batch=B, max_seq=S, device=local, flags=args.flags)
        self.enc_t = rlx.Encoder.from_config(cfg, max_batch=B, max_seq=S, device=local, flags=args.flags | binding.FLAG_KERNEL_EVENTS)
        self.ws, self.ws_t = self.enc.alloc_workspace(B, S), self.enc_t.alloc_workspace(B, S)
        self.ids_d = torch.from_numpy(self.mine.ids).cuda()
        self.mask_d = torch.from_numpy(self.mine.mask).cuda()
        self.out_d = torch.empty((B, H), dtype=torch.float32, device="cuda")
        self.ids_h = torch.from_numpy(self.mine.ids).pin_memory()
        self.mask_h = torch.from_numpy(self.mine.mask).pin_memory()
        self.out_h = torch.empty((B, H), dtype=torch.float32).pin_memory()
        self.flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        self.n_kernels = self.enc.kernels_per_forward(B, S)
        per_layer = (self.n_kernels - 3) // cfg.num_layers
        # 7 = plain layer; 5 = both LayerNorms fused into the GEMMs; 3 = QKV GEMM, attention, one kernel for the rest
        fused_ffn = per_layer == 3
        self.names = kernel_classes(cfg.num_layers, fused_ln=(per_layer == 5), fused_ffn=fused_ffn)
        assert len(self.names) == self.n_kernels

    def step_device(self, e, w):
        torch = self.torch
        with torch.cuda.stream(self.stream):
            self.flush.zero_()                      # evict L2 (256 MiB > 126 MB)
            t0 = torch.cuda.Event(enable_timing=True)
            t1 = torch.cuda.Event(enable_timing=True)
            t0.record(self.stream)
            e.forward(self.ids_d, self.mask_d, self.weights, self.out_d, w, stream=self.stream)
            t1.record(self.stream)
        return t0, t1

    def warm(self, n, e2e=True):
        for _ in range(n):
            self.step_device(self.enc, self.ws)
            self.step_device(self.enc_t, self.ws_t)
            if e2e:
                with self.torch.cuda.stream(self.stream):
                    self.enc.forward_host(self.ids_h, self.mask_h, self.weights, self.out_h, self.ws, stream=self.stream)

    def timed_device(self, steps):
        return [self.step_device(self.enc, self.ws) for _ in range(steps)]

    def timed_e2e(self, steps):
        ms = []
        for _ in range(steps):
            with self.torch.cuda.stream(self.stream):
                self.flush.zero_()
            self.stream.synchronize()
            t0 = time.perf_counter()
            self.enc.forward_host(self.ids_h, self.mask_h, self.weights, self.out_h, self.ws, stream=self.stream)   # syncs itself
            ms.append((time.perf_counter() - t0) * 1e3)
        return ms

    def timed_kernels(self, steps):
        per_class = {}
        B, S = self.cfg.batch, self.cfg.seq
        for _ in range(steps):
            self.step_device(self.enc_t, self.ws_t)
            for n, t in zip(self.names, self.enc_t.kernel_times(B, S)):
                per_class.setdefault(n, []).append(t)
        return per_class

    def close(self):
        self.enc.close()
        self.enc_t.close()


def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2609_37916_b200.build import build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build()
    if world > 1:
        dist.barrier()

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    run = EncoderRun(args.config, args, rank, local)
    cfg, B, S, H = run.cfg, run.cfg.batch, run.cfg.seq, run.cfg.hidden
    warmup = max(args.warmup, 3)
    run.warm(warmup)          # also captures the graphs
    barrier()
    assert run.enc.last_device_status(run.ws, stream=run.stream) == 0

    sampler = ClockSampler(local)
    sampler.start()

    # ---- timed region 1: K graph replays, device-resident inputs ----
    barrier()
    sampler.active.set()
    wall0 = time.perf_counter()
    evs = run.timed_device(args.steps)
    barrier()
    wall1 = time.perf_counter()
    step_ms = [a.elapsed_time(b) for a, b in evs]
    # ---- timed region 2: end to end through the host-buffer entry point ----
    e2e_ms = run.timed_e2e(args.steps)
    barrier()
    # ---- timed region 3: event-node intervals (used to split the step time among the kernels) ----
    per_class = run.timed_kernels(args.steps)
    barrier()
    sampler.active.clear()
    sampler.stop()
    status = run.enc.last_device_status(run.ws, stream=run.stream)

    # ---- reduce over ranks (max of times) ----
    total_ms, e2e_total = sum(step_ms), sum(e2e_ms)
    red = torch.tensor([total_ms, e2e_total, statistics.median(step_ms), statistics.median(e2e_ms)],
                       dtype=torch.float64, device="cuda")
    if world > 1:
        dist.all_reduce(red, op=dist.ReduceOp.MAX)
    total_ms, e2e_total, p50_ms, e2e_p50 = [float(v) for v in red.cpu()]

    # ---- the roofline configuration rides along with the default (headline) run ----
    roofline_c3 = None
    if rank == 0 and world == 1 and args.config == "c2" and not args.no_c3:
        run3 = EncoderRun("c3", args, 0, local)
        run3.warm(3, e2e=False)
        torch.cuda.synchronize()
        s3 = ClockSampler(local)
        s3.start()
        s3.active.set()
        ev3 = run3.timed_device(args.c3_steps)
        torch.cuda.synchronize()
        pc3 = run3.timed_kernels(args.c3_steps)
        torch.cuda.synchronize()
        s3.active.clear()
        s3.stop()
        ms3 = [a.elapsed_time(b) for a, b in ev3]
        peaks3, kind3 = load_peaks()
        kt3, ov3 = kernel_table(run3.cfg, run3.mine.lengths, run3.names, pc3, statistics.median(ms3), peaks3)
        for cls, mb in load_dram_traffic().get("c3", {}).items():   # ncu dram__bytes per launch (profiles/dram_traffic.md)
            if cls in kt3:
                kt3[cls]["traffic"] = mb * 1e6
        roofline_c3 = {"workload": workload_config("c3")["workload"], "steps": args.c3_steps, "p50_ms": statistics.median(ms3),
                       "sequences_per_s": run3.cfg.batch / (statistics.median(ms3) / 1e3), "valid_tokens": int(run3.mine.lengths.sum()),
                       "clocks": s3.summary(), "peak_source": kind3, "event_overhead_us_per_launch": ov3,
                       "kernels": {k: {f: (round(v, 4) if isinstance(v, float) else v) for f, v in row.items()} for k, row in kt3.items()},
                       "device_status": run3.enc.last_device_status(run3.ws, stream=run3.stream)}
        run3.close()
        del run3
        torch.cuda.empty_cache()

    if rank == 0:
        peaks, peak_kind = load_peaks()
        gpu_busy_s = total_ms / 1e3
        ktab, overhead_us = kernel_table(cfg, run.mine.lengths, run.names, per_class, p50_ms, peaks)
        dom = max(ktab, key=lambda k: ktab[k]["ms_per_step"])
        d = ktab[dom]
        traffic_mb = load_dram_traffic().get(args.config, {}).get(dom)
        roofline = {"kernel": dom, "bound": d["bound"], "achieved": d["achieved"], "peak": d["peak"], "unit": d["unit"],
                    "frac": d["frac"], "traffic": None if traffic_mb is None else traffic_mb * 1e6,
                    "traffic_source": "profiles/dram_traffic.md (ncu dram__bytes per launch)",
                    "peak_source": f"{peak_kind} (burst: kernels are timed one by one inside a sub-millisecond step)",
                    "share_of_step": d["share"],
                    "timing": "untouched graph replay (programmatic dependent launch on) split among the kernels in "
                              "proportion to their event-node intervals",
                    "event_interval_us": d["event_interval_us"], "event_overhead_us_per_launch": overhead_us}

        cb = time_oracle(args.config, budget_s=12.0, steps=1, all_valid=args.all_valid)
        cb_value = cb["n"] / cb["times"][0]
        # the oracle's embeddings of its sample double as a parity check of this very run (rank 0's batch)
        n = cb["n"]
        got = run.out_d[:n].double().cpu().numpy()
        keep = run.mine.lengths[:n] > 0

        def compare(ref):
            cos = (got * ref).sum(1)[keep] / np.maximum(np.linalg.norm(got, axis=1) * np.linalg.norm(ref, axis=1), 1e-300)[keep]
            return {"min_cosine": float(cos.min()) if cos.size else None, "max_abs_err": float(np.abs(got - ref).max())}

        parity = {"sequences": int(n), **compare(cb["embeddings"])}
        # secondary reading of the weight precision: the oracle on the UNROUNDED fp32 draws (the GPU always
        # holds their bf16 roundings), reported next to the primary one, not gated
        from oracle import oracle
        from synth.inputs import EncoderConfig, make_inputs
        n2 = max(1, min(n, int(n * 8.0 / max(cb["times"][0], 1e-3))))
        raw = make_inputs(cfg, fp32_weights=True, lengths=np.full(cfg.batch, cfg.seq, dtype=np.int64) if args.all_valid else None)
        ref2 = oracle.encoder_forward(EncoderConfig(**{**cfg.__dict__, "batch": n2}), raw.ids[:n2], raw.mask[:n2], raw.params, raw.layers)
        got2, keep2 = got[:n2], keep[:n2]
        cos2 = (got2 * ref2).sum(1)[keep2] / np.maximum(np.linalg.norm(got2, axis=1) * np.linalg.norm(ref2, axis=1), 1e-300)[keep2]
        parity["fp32_weight_oracle"] = {"sequences": int(n2), "min_cosine": float(cos2.min()) if cos2.size else None,
                                        "max_abs_err": float(np.abs(got2 - ref2).max())}
        seqs = B * world
        line = {
            "metric": METRIC, "value": seqs * args.steps / (total_ms / 1e3), "unit": "sequences/s",
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": total_ms / args.steps,
            "p50_ms": p50_ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": workload_config(args.config, {"valid_lengths": f"all {cfg.seq} (--all-valid)"} if args.all_valid else None),
            "e2e": {"value": seqs * args.steps / (e2e_total / 1e3), "unit": "sequences/s", "p50_ms": e2e_p50,
                    "h2d_bytes_per_step": 2 * B * S * 4, "d2h_bytes_per_step": B * H * 4,
                    "timing": "host wall clock around rlx_encoder_forward_host with pinned host buffers: the kernels read ids / mask from, and write the embeddings to, host memory over the bus (no separate copy operations), then the stream is synchronised"},
            # main chain + the side-branch weight prefetch kernel (models whose Linear weights fit in L2)
            "gpu_launches": args.steps * (run.n_kernels + (1 if cfg.num_layers * 24 * cfg.hidden * cfg.hidden <= (48 << 20)
                                                           and cfg.ffn == 4 * cfg.hidden else 0)),
            "clocks": sampler.summary(),
            "roofline": roofline,
            "kernels": ktab,
            "cpu_baseline": {"value": cb_value, "unit": "sequences/s", "cores": cb["cores"], "kind": "oracle",
                             "sample": f"first {cb['n']} of {cb['batch']} sequences of {args.config}, 1 run, "
                                       f"{cb['times'][0]:.2f} s"},
            "context": {"paper_p50_ms_batch32_seq128": {"RLX-Metal": 16.6, "PyTorch-MPS": 26.74,
                                                        "hardware": "one Apple Silicon host (paper Section 8.1)"}},
            "parity_on_sample": parity,
            "device_status": status,
            "wall_s_timed_region": wall1 - wall0,
            "gpu_busy_s": gpu_busy_s,
        }
        if roofline_c3 is not None:
            line["roofline_c3"] = roofline_c3
        print(json.dumps(line), flush=True)
    run.close()
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# ---------------------------------------------------------------------------- attention under other mask kinds
def attention_kind_workload(seed: int = 7, batch: int = 16, lo: int = 1024, hi: int = 4096):
    rng = np.random.default_rng(seed)
    return rng.integers(lo, hi + 1, size=batch).astype(np.int32)


def visible_pairs(lengths, kind: str, window: int) -> int:
    tot = 0
    for n in (int(x) for x in lengths):
        if kind == "none":
            tot += n * n
        elif kind == "causal":
            tot += n * (n + 1) // 2
        else:
            i = np.arange(n, dtype=np.int64)
            tot += int(np.minimum(i + 1, window).sum())
    return tot


def run_attention_kind(args):
    """`--op attention_kind`: one step = one launch of rlx_attention_kind_bf16 over a packed batch of
    decoder-shaped sequences (16 heads x 64, lengths 1024..4096, seeded), device-timed with an L2 flush
    between steps; the oracle is timed on the first sequence."""
    import torch
    import paper_2609_37916_b200 as rlx

    h, d = args.heads, args.head_dim
    hkv = args.kv_heads or h
    H = h * d
    lengths = attention_kind_workload()
    total, max_len = int(lengths.sum()), int(lengths.max())
    start = np.concatenate([[0], np.cumsum(lengths)])[:-1].astype(np.int32)
    kind_id = {"none": rlx.binding.MASK_NONE, "causal": rlx.binding.MASK_CAUSAL, "sliding": rlx.binding.MASK_SLIDING_WINDOW}[args.mask]
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(7)
    qkv = torch.randn(total, (h + 2 * hkv) * d, device="cuda", generator=g).to(torch.bfloat16)
    ss, sl = torch.from_numpy(start).cuda(), torch.from_numpy(lengths).cuda()
    rope = rlx.rope_tables(max_len, d) if args.rope else None
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    ctx = torch.zeros(total, H, dtype=torch.bfloat16, device="cuda")
    sampler = ClockSampler(0)
    sampler.start()

    def step():
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = rlx.binding.attention_kind_bf16(qkv, ss, sl, max_len, h, kind_id, args.window, rope, out=ctx, num_kv_heads=hkv)
        e1.record()
        return e0, e1, out

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler.active.set()
    evs = [step() for _ in range(args.steps)]
    torch.cuda.synchronize()
    sampler.active.clear()
    sampler.stop()
    ms = [a.elapsed_time(b) for a, b, _ in evs]
    p50 = statistics.median(ms)
    pairs = visible_pairs(lengths, args.mask, args.window)
    flops, exps, bytes_ = 4.0 * pairs * d * h, float(pairs) * h, 2.0 * total * (2 * h + 2 * hkv) * d
    peaks, peak_kind = load_peaks()
    # oracle on the first sequence
    from oracle import attention_kinds as ak
    n0 = int(lengths[0])
    seq = qkv[:n0].float().cpu().numpy().astype(np.float64)
    t0 = time.perf_counter()
    ref = ak.attention_one(seq, h, kind_id, args.window, 10000.0 if args.rope else None, num_kv_heads=hkv)
    t_or = time.perf_counter() - t0
    got = evs[-1][2][:n0].float().cpu().numpy().astype(np.float64)
    line = {
        "metric": "attention (mask kind / rotary) tokens/s (p50 ms reported alongside)", "op": "attention_kind",
        "value": total * args.steps / (sum(ms) / 1e3), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sum(ms) / args.steps, "p50_ms": p50, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"packed batch of 16 sequences, lengths 1024..4096 (seed 7, {total} tokens), {h} q heads / {hkv} kv heads x {d}, "
                               f"mask {args.mask}" + (f"({args.window})" if args.mask == "sliding" else "") +
                               (", rotary q,k" if args.rope else ""), "l2": "256 MiB flush write between steps"},
        "gpu_launches": args.steps, "clocks": sampler.summary(),
        "roofline": {"kernel": f"attention_bf16_kernel<{d}>", "bound": "alu", "achieved": exps / (p50 * 1e-3) / 1e12,
                     "peak": EXP_PEAK_TEXP_S, "unit": "Texp/s", "frac": exps / (p50 * 1e-3) / 1e12 / EXP_PEAK_TEXP_S,
                     "traffic": None, "tensor_tflops": flops / (p50 * 1e-3) / 1e12,
                     "tensor_frac_of_" + peak_kind: flops / (p50 * 1e-3) / 1e12 / peaks["bf16_tflops"],
                     "hbm_gbs": bytes_ / (p50 * 1e-3) / 1e9,
                     "work": "visible (query, key) pairs only"},
        "cpu_baseline": {"value": n0 / t_or, "unit": "tokens/s", "cores": usable_cores(), "kind": "oracle",
                         "sample": f"first sequence ({n0} tokens), 1 run, {t_or:.2f} s"},
        "parity_on_sample": {"max_abs_err": float(np.abs(got - ref).max()), "max_abs_ref": float(np.abs(ref).max())},
    }
    print(json.dumps(line), flush=True)


def run_qk_rope(args):
    """`--op qk_rope`: one step = one launch of rlx_qk_rope_bf16 (in-place rotation of the q and k column
    blocks) over the packed batch of `--op attention_kind`; HBM-bound: 2/3 of qkv read and written."""
    import torch
    import paper_2609_37916_b200 as rlx

    h, d = 16, 64
    H = h * d
    lengths = attention_kind_workload()
    total, max_len = int(lengths.sum()), int(lengths.max())
    start = np.concatenate([[0], np.cumsum(lengths)])[:-1].astype(np.int32)
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(7)
    qkv0 = torch.randn(total, 3 * H, device="cuda", generator=g).to(torch.bfloat16)
    qkv = qkv0.clone()
    ss, sl = torch.from_numpy(start).cuda(), torch.from_numpy(lengths).cuda()
    rope = rlx.rope_tables(max_len, d)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    sampler = ClockSampler(0)
    sampler.start()

    def step():
        qkv.copy_(qkv0)          # keep magnitudes fixed: the rotation is applied to fresh data every step
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rlx.binding.qk_rope_bf16(qkv, ss, sl, max_len, h, rope)
        e1.record()
        return e0, e1

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler.active.set()
    evs = [step() for _ in range(args.steps)]
    torch.cuda.synchronize()
    sampler.active.clear()
    sampler.stop()
    ms = [a.elapsed_time(b) for a, b in evs]
    p50 = statistics.median(ms)
    bytes_ = 2.0 * total * 2 * H * 2          # q and k blocks, read and written, bf16
    peaks, peak_kind = load_peaks()
    from oracle import attention_kinds as ak
    n0 = int(lengths[0])
    t0 = time.perf_counter()
    ref = ak.rope_qk_packed(qkv0[:n0].float().cpu().numpy().astype(np.float64), [0], [n0], h, 10000.0)
    t_or = time.perf_counter() - t0
    got = qkv[:n0].float().cpu().numpy().astype(np.float64)
    ach = bytes_ / (p50 * 1e-3) / 1e9
    line = {
        "metric": "fused QK-RoPE tokens/s (p50 ms reported alongside)", "op": "qk_rope",
        "value": total * args.steps / (sum(ms) / 1e3), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sum(ms) / args.steps, "p50_ms": p50, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"packed batch of 16 sequences, lengths 1024..4096 (seed 7, {total} tokens), 16 heads x 64",
                   "l2": "256 MiB flush write between steps"},
        "gpu_launches": args.steps, "clocks": sampler.summary(),
        "roofline": {"kernel": "qk_rope_kernel<64>", "bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": ach / peaks["hbm_gbs"], "traffic": None, "peak_source": peak_kind},
        "cpu_baseline": {"value": n0 / t_or, "unit": "tokens/s", "cores": usable_cores(), "kind": "oracle",
                         "sample": f"first sequence ({n0} tokens), 1 run, {t_or:.3f} s"},
        "parity_on_sample": {"max_abs_err": float(np.abs(got - ref).max()), "max_abs_ref": float(np.abs(ref).max())},
    }
    print(json.dumps(line), flush=True)


def run_mx_matmul(args):
    """`--op mx_matmul`: the block-scaled tensor-core path (both operands FP8 E4M3 with E8M0 scales per 32) on the
    encoder's three projection shapes at the roofline configuration's row count and on a large square problem;
    the activation quantiser is timed alone.  The JSON line's value / roofline are the FFN-down shape's."""
    import torch
    import paper_2609_37916_b200 as rlx
    from oracle import scaled_matmul as osm

    torch.cuda.set_device(0)
    word = rlx.binding.FMT_FP8_E4M3
    g = torch.Generator(device="cuda").manual_seed(5)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    peaks, peak_kind = load_peaks()
    fp8_peak = 2.0 * peaks["bf16_tflops"]
    sampler = ClockSampler(0)
    sampler.start()
    shapes = [("qkv", 36736, 1152, 384), ("ffn_up", 36736, 1536, 384), ("ffn_down", 36736, 384, 1536), ("square", 8192, 8192, 8192)]
    rows = {}
    first = True
    for name, M, N, K in shapes:
        x = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
        w = (torch.randn(N, K, device="cuda", generator=g) * 0.05).to(torch.bfloat16)
        bias = torch.randn(N, device="cuda", generator=g)
        a_codes, a_scales = rlx.quantise_mx(x, word)
        w_codes, w_scales = rlx.quantise_mx(w, word)      # weights through the same rule (bit-exact against the oracle's)
        out = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")

        def timed(fn):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            return e0, e1

        mm = lambda: rlx.mx_matmul_bf16(a_codes, a_scales, word, w_codes, w_scales, word, bias=bias, out=out)
        qz = lambda: rlx.quantise_mx(x, word)
        for _ in range(max(args.warmup, 3)):
            timed(mm)
            timed(qz)
        torch.cuda.synchronize()
        if first:
            sampler.active.set()
        ev = [timed(mm) for _ in range(args.steps)]
        evq = [timed(qz) for _ in range(args.steps)]
        torch.cuda.synchronize()
        ms = statistics.median(a.elapsed_time(b) for a, b in ev)
        msq = statistics.median(a.elapsed_time(b) for a, b in evq)
        tf = 2.0 * M * N * K / (ms * 1e-3) / 1e12
        hbm_floor_us = (M * K + N * K + (M + N) * K / 32 + 2.0 * M * N) / (peaks["hbm_gbs"] * 1e9) * 1e6
        rows[name] = {"M": M, "N": N, "K": K, "p50_us": ms * 1e3, "tflops": tf, "frac_of_fp8_peak": tf / fp8_peak,
                      "hbm_floor_us": hbm_floor_us, "tensor_floor_us": 2.0 * M * N * K / (fp8_peak * 1e12) * 1e6,
                      "quantise_p50_us": msq * 1e3, "quantise_gbs": M * K * (2 + 1 + 1 / 32) / (msq * 1e-3) / 1e9}
        if name == "ffn_down":
            m0 = 64     # parity of the timed launch's output on a sample, against the fp64 product of the dequantised operands
            ref = osm.mx_matmul(a_codes[:m0].cpu().numpy(), a_scales[:m0].cpu().numpy(), osm.E4M3, w_codes.cpu().numpy(),
                                w_scales.cpu().numpy(), osm.E4M3, bias.cpu().numpy().astype(np.float64))
            got = out[:m0].float().cpu().numpy().astype(np.float64)
            rows[name]["max_err_over_max_ref"] = float(np.abs(got - ref).max() / np.abs(ref).max())
        first = False
    sampler.active.clear()
    sampler.stop()
    r = rows["ffn_down"]
    line = {
        "metric": "block-scaled FP8 matmul tokens/s (p50 reported alongside)", "op": "mx_matmul",
        "value": r["M"] / (r["p50_us"] * 1e-6), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": r["p50_us"] * 1e-3, "p50_ms": r["p50_us"] * 1e-3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "fp8_e4m3 x fp8_e4m3 -> f32 accumulate -> bf16",
        "data": "synthetic",
        "config": {"workload": "M=36736 tokens, N=384, K=1536 (FFN-down shape), both operands FP8 E4M3 with E8M0 scales per 32; "
                               "the other shapes are in `shapes`", "l2": "256 MiB flush write between steps"},
        "gpu_launches": args.steps, "clocks": sampler.summary(),
        "roofline": {"kernel": "gemm_mx192_tcgen05_kernel", "bound": "tensor", "achieved": r["tflops"], "peak": fp8_peak,
                     "unit": "TFLOP/s", "frac": r["frac_of_fp8_peak"], "traffic": None,
                     "peak_source": peak_kind + "; FP8 peak taken as 2 x the measured bf16 figure (no FP8 peak measured)"},
        "e2e": None, "cpu_baseline": None, "shapes": rows,
    }
    print(json.dumps(line))


def run_scaled_matmul(args):
    """`--op scaled_matmul`: one step = rlx_scaled_matmul_bf16 (block-scaled minifloat weights dequantised
    to bf16, then the tcgen05 GEMM with bias) at the BERT-base FFN-up shape over 32,768 tokens; the
    dequantisation pass is also timed alone on a matrix larger than L2."""
    import torch
    import paper_2609_37916_b200 as rlx
    from synth.inputs import make_block_scaled_weights, pack_nibbles

    fmts = {"fp8_e4m3": (rlx.binding.FMT_FP8_E4M3, 8, 0x7E, False, "E4M3"), "fp4_e2m1": (rlx.binding.FMT_FP4_E2M1, 4, 7, True, "E2M1")}
    word, bits, maxmag, packed, oname = fmts[args.fmt]
    M, N, K = 32768, 3072, 768
    torch.cuda.set_device(0)
    g = torch.Generator(device="cuda").manual_seed(3)
    a = torch.randn(M, K, device="cuda", generator=g).to(torch.bfloat16)
    bias = torch.randn(N, device="cuda", generator=g)
    codes, scales = make_block_scaled_weights(3, N, K, bits, maxmag, 122, 128)
    dev_codes = torch.from_numpy(pack_nibbles(codes) if packed else codes).cuda()
    dev_scales = torch.from_numpy(scales).cuda()
    w_scratch = torch.empty(N, K, dtype=torch.bfloat16, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    # the big matrix for the dequantisation pass alone
    N2, K2 = 16384, 8192
    codes2, scales2 = make_block_scaled_weights(4, N2, K2, bits, maxmag, 122, 128)
    dev_codes2 = torch.from_numpy(pack_nibbles(codes2) if packed else codes2).cuda()
    dev_scales2 = torch.from_numpy(scales2).cuda()
    w2 = torch.empty(N2, K2, dtype=torch.bfloat16, device="cuda")
    sampler = ClockSampler(0)
    sampler.start()

    def timed(fn):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        out = fn()
        e1.record()
        return e0, e1, out

    y = torch.empty(M, N, dtype=torch.bfloat16, device="cuda")
    mm = lambda: rlx.scaled_matmul_bf16(a, dev_codes, dev_scales, word, bias, w_scratch=w_scratch, out=y)
    dq = lambda: rlx.dequant_block_scaled_bf16(dev_codes2, dev_scales2, N2, K2, word, out=w2)
    for _ in range(max(args.warmup, 3)):
        timed(mm)
        timed(dq)
    torch.cuda.synchronize()
    sampler.active.set()
    ev_mm = [timed(mm) for _ in range(args.steps)]
    ev_dq = [timed(dq) for _ in range(args.steps)]
    torch.cuda.synchronize()
    sampler.active.clear()
    sampler.stop()
    ms = [x.elapsed_time(y) for x, y, _ in ev_mm]
    ms_dq = [x.elapsed_time(y) for x, y, _ in ev_dq]
    p50, p50_dq = statistics.median(ms), statistics.median(ms_dq)
    peaks, peak_kind = load_peaks()
    flops = 2.0 * M * N * K
    dq_bytes = N2 * K2 * (0.5 if packed else 1.0) + N2 * K2 / 32 + 2.0 * N2 * K2
    # oracle: fp64 matmul on the dequantised grid for the first rows
    from oracle import scaled_matmul as osm
    m0 = 256
    t0 = time.perf_counter()
    ref = osm.scaled_matmul(a[:m0].float().cpu().numpy().astype(np.float64), codes, scales, getattr(osm, oname),
                            bias.cpu().numpy().astype(np.float64))
    t_or = time.perf_counter() - t0
    got = ev_mm[-1][2][:m0].float().cpu().numpy().astype(np.float64)
    ach = flops / (p50 * 1e-3) / 1e12
    line = {
        "metric": "ScaledMatMul tokens/s (p50 ms reported alongside)", "op": "scaled_matmul",
        "value": M * args.steps / (sum(ms) / 1e3), "unit": "tokens/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sum(ms) / args.steps, "p50_ms": p50, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"M={M} tokens, N={N}, K={K} (BERT-base FFN-up), weights {args.fmt} with E8M0 scales per 32, "
                               "dequantise + GEMM(+bias) per step", "l2": "256 MiB flush write between steps"},
        "gpu_launches": 2 * args.steps, "clocks": sampler.summary(),
        "roofline": {"kernel": "gemm_tcgen05_kernel", "bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops"],
                     "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops"], "traffic": None, "peak_source": peak_kind,
                     "note": "interval = dequantisation pass + GEMM"},
        "dequant": {"workload": f"{N2} x {K2} weights", "p50_ms": p50_dq, "bound": "hbm",
                    "achieved": dq_bytes / (p50_dq * 1e-3) / 1e9, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                    "frac": dq_bytes / (p50_dq * 1e-3) / 1e9 / peaks["hbm_gbs"]},
        "cpu_baseline": {"value": m0 / t_or, "unit": "tokens/s", "cores": usable_cores(), "kind": "oracle",
                         "sample": f"first {m0} rows, 1 run, {t_or:.2f} s"},
        "parity_on_sample": {"max_abs_err": float(np.abs(got - ref).max()), "max_abs_ref": float(np.abs(ref).max())},
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="c2", choices=["c0", "c1", "c2", "c3", "c4"])
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--flags", type=lambda v: int(v, 0), default=0, help="encoder op: rlx_encoder_config_t.flags (e.g. 0x200)")
    ap.add_argument("--all-valid", action="store_true", help="encoder op: every sequence has the full length")
    ap.add_argument("--no-c3", action="store_true", help="encoder op, default workload: skip the roofline_c3 block")
    ap.add_argument("--c3-steps", type=int, default=20, help="timed steps of the roofline_c3 block")
    ap.add_argument("--op", default="encoder", choices=["encoder", "attention_kind", "qk_rope", "scaled_matmul", "mx_matmul"])
    ap.add_argument("--fmt", default="fp8_e4m3", choices=["fp8_e4m3", "fp4_e2m1"])
    ap.add_argument("--mask", default="causal", choices=["none", "causal", "sliding"])
    ap.add_argument("--window", type=int, default=512)
    ap.add_argument("--rope", type=int, default=1)
    ap.add_argument("--heads", type=int, default=16, help="attention_kind op: q heads (head_dim 64)")
    ap.add_argument("--head-dim", type=int, default=64, choices=[32, 64, 128], help="attention_kind op: head size")
    ap.add_argument("--kv-heads", type=int, default=0, help="attention_kind op: k/v heads (0 = same as --heads)")
    args = ap.parse_args()
    if args.op != "encoder":
        if args.impl != "ours" or args.gpus != 1:
            raise SystemExit(f"--op {args.op} runs on one GPU with --impl ours")
        {"attention_kind": run_attention_kind, "qk_rope": run_qk_rope, "scaled_matmul": run_scaled_matmul,
         "mx_matmul": run_mx_matmul}[args.op](args)
        return
    if args.impl == "reference":
        run_reference_arm(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

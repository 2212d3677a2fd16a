#!/usr/bin/env python
"""Benchmark of the SQuat KV-cache write path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl reference]

One "step" is one pass of the whole write path over one layer-batch of synthetic input:
subspace build (Gram, eigen-decomposition, update matrices) -> key quantization -> value
quantization -> dequantization of both (the read-back).  Default workload: config 1, the
Llama-2-7B-shaped layer (32 heads x 4096 tokens x 128, bf16, r = 32, 2 bits, G = 32).
Workload 3 (--config 3) is the decode-append stream: the subspace is built from the 2048-token prompt, then
32 windows of [64, 32, 128, 128] keys and values are appended, one call of each quantizer per window, into a
4096-token cache that is dequantized at the end; the line then also carries per-call latencies.
Inputs are resident in HBM before the timed region; L2 is flushed between steps; every step
and every stage is timed with CUDA events on the launching stream; with N > 1 ranks each
rank processes its own replica of the workload (the path has no exchange step) and the
slowest rank's time counts.  Prints ONE JSON line on rank 0.

`--impl reference` times the CPU oracle (plain single-threaded fp64 C, as it stands) on a bounded
sample of the same workload.
"""
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

import numpy as np  # noqa: E402

import squat_inputs as si  # noqa: E402

METRIC = "key vectors quantized/sec (whole write path: subspace build + keys + values + dequantize)"
UNIT = "key_vectors/s"

# Nominal FP32 peak of a B200: 148 SMs x 128 FMA lanes x 2 flop x 1.965 GHz (max SM clock).  Context only: the
# roofline uses the figure the probe kernel reaches in this run (measure_fp32_peak).
SM_COUNT, FMA_LANES, SM_MAX_GHZ = 148, 128, 1.965
ALU_PEAK_TFLOPS = SM_COUNT * FMA_LANES * 2 * SM_MAX_GHZ / 1e3

TRAFFIC_FILE = os.path.join(ROOT, "profiles", "quant_keys_kernel_traffic.json")


def key_kernel_traffic(cfg, args):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of the key kernel on this workload, from the tracked
    summary of an ncu capture (which names the source revision it was taken on); None where no capture covers it."""
    try:
        with open(TRAFFIC_FILE) as f:
            rec = json.load(f)
    except (OSError, ValueError):
        return None
    key = "config %d b=%d r=%d G=%d%s" % (cfg.index, cfg.bits, cfg.rank_r, cfg.group_size, " m16" if args.meta16 else "")
    ent = rec.get("workloads", {}).get(key)
    if not ent:
        return None
    return {"dram_bytes_per_launch": ent["dram_bytes_per_launch"], "captured_at_commit": rec.get("commit"),
            "note": ent.get("note")}


def measure_fp32_peak(sq, dev):
    """FP32 multiply-add throughput this GPU reaches on the library's probe kernel (scalar and two-wide forms), timed
    with CUDA events before the benchmark's timed region; the roofline quotes the better of the two."""
    import torch
    sink = torch.zeros(4, dtype=torch.float32, device=dev)
    stream = torch.cuda.current_stream()
    out = {}
    for name, packed in (("fma_f32", False), ("fma_f32x2", True)):
        best = 0.0
        for it in range(7):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            flops = sq.squat_fp32_peak_probe(packed, 2048 if packed else 4096, sink)
            b.record(stream)
            torch.cuda.synchronize()
            if it >= 2:
                best = max(best, flops / (a.elapsed_time(b) * 1e-3) / 1e12)
        out[name + "_tflops"] = best
    out["tflops"] = max(out["fma_f32_tflops"], out["fma_f32x2_tflops"])
    return out


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d.get("bf16_tflops", 1590.0), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


# --------------------------------------------------------------------------- algorithmic counts
def key_flops_per_vector(d, g, r=None):
    """2 x FMAs of the update per key vector: the dense block-triangular form (Eq. (3) / Eq. (update_block)) or, if
    cheaper, the rank-r form of the same update (2 r d FMAs) -- the algorithmic count is the smaller of the two,
    whichever of them a kernel runs."""
    T = d // g
    tri = sum(g * (d - t * g) for t in range(1, T))
    return 2 * (tri if r is None else min(tri, 2 * r * d))


def key_fma_split(d, g, blk=32):
    """The same multiply-adds split by where the key kernel runs them: (inside a 32-channel block: FP32 pipes,
    across blocks: tensor cores).  W[j'][j] is non-zero iff j' lies in a later g-block than j."""
    alu = sum(1 for j in range(d) for jp in range(j + 1, d) if jp // g > j // g and jp // blk == j // blk)
    tensor = sum(1 for j in range(d) for jp in range(j + 1, d) if jp // g > j // g and jp // blk != j // blk)
    return alu, tensor


def reader_bytes_per_cached_token(d, bits, G, meta_bytes=4):
    """What one decode step has to read per cached token: key and value codes, key metadata (scale and zero per
    channel, shared by G tokens), value metadata (scale and zero per group of G channels); metadata float32 or
    binary16."""
    return 2 * d * bits // 8 + 2 * meta_bytes * d // G + 2 * meta_bytes * d // G


def bytes_per_vector(d, bits, G, elem_bytes, meta_bytes=4):
    """Algorithmic HBM bytes per key (or value) vector: read the vector, write codes + scale and zero (float32, or
    binary16 for the 16-bit-metadata cache)."""
    return d * elem_bytes + d * bits // 8 + 2 * meta_bytes * d // G


# --------------------------------------------------------------------------- clocks sampling
class ClockSampler:
    """Samples SM clock and throttle reasons while the timed region runs: NVML polled every 2 ms from a thread
    (read-only queries), or, where the NVML binding is missing, nvidia-smi at its 100 ms cadence."""
    FIELDS = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
              "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, gpu_index, pci_bus_id=None):
        self.gpu_index, self.pci_bus_id = gpu_index, pci_bus_id
        self.proc, self.lines = None, []
        self.nvml, self.handle, self.thread, self.stop_flag = None, None, None, threading.Event()
        self.sm, self.mx, self.reasons = [], [], set()
        self.errors, self.last_error = 0, None

    def _nvml_open(self):
        try:
            import pynvml
            pynvml.nvmlInit()
            if self.pci_bus_id:
                try:
                    self.handle = pynvml.nvmlDeviceGetHandleByPciBusId(self.pci_bus_id.encode())
                except pynvml.NVMLError:
                    self.handle = None
            if self.handle is None:
                self.handle = pynvml.nvmlDeviceGetHandleByIndex(self.gpu_index)
            self.nvml = pynvml
            return True
        except Exception:
            self.nvml = None
            return False

    def _nvml_poll(self):
        n = self.nvml
        masks = {"hw_slowdown": n.nvmlClocksEventReasonHwSlowdown if hasattr(n, "nvmlClocksEventReasonHwSlowdown") else 0x8,
                 "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
        get_reasons = getattr(n, "nvmlDeviceGetCurrentClocksEventReasons", None) or n.nvmlDeviceGetCurrentClocksThrottleReasons
        try:
            mx = n.nvmlDeviceGetMaxClockInfo(self.handle, n.NVML_CLOCK_SM)
        except n.NVMLError:
            mx = None
        while not self.stop_flag.is_set():
            try:
                self.sm.append(float(n.nvmlDeviceGetClockInfo(self.handle, n.NVML_CLOCK_SM)))
                if mx:
                    self.mx.append(float(mx))
                r = int(get_reasons(self.handle))
                for name, bit in masks.items():
                    if r & bit:
                        self.reasons.add(name)
            except n.NVMLError as e:
                self.errors += 1
                self.last_error = str(e)
            time.sleep(0.001)

    def start(self):
        if self._nvml_open():
            try:                               # the first query of a process is slow (lazy initialisation): pay for it here
                self.nvml.nvmlDeviceGetClockInfo(self.handle, self.nvml.NVML_CLOCK_SM)
            except Exception as e:
                self.last_error = str(e)
            self.thread = threading.Thread(target=self._nvml_poll, daemon=True)
            self.thread.start()
            return
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-i", str(self.gpu_index), "-lms", "100"], stdout=subprocess.PIPE,
                                         stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._pump, daemon=True).start()
        except OSError:
            self.proc = None

    def _pump(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join(timeout=1)
            try:
                self.nvml.nvmlShutdown()
            except Exception:
                pass
            out = {"sm_mhz": statistics.median(self.sm) if self.sm else None, "sm_max_mhz": max(self.mx) if self.mx else None,
                   "samples": len(self.sm), "source": "nvml", "reasons": sorted(self.reasons)}
            if self.errors:
                out["query_errors"], out["last_error"] = self.errors, self.last_error
            return out
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "source": "nvidia-smi", "reasons": sorted(reasons)}


# --------------------------------------------------------------------------- distributed glue
def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


def aggregate_over_ranks(local_ms, local_units, device=None):
    """Whole-job figures: time = max over ranks, units = sum over ranks.  Works on any backend."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return local_ms, local_units
    t = torch.tensor([local_ms], dtype=torch.float64, device=device)
    u = torch.tensor([float(local_units)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), int(round(u.item()))


# --------------------------------------------------------------------------- the CPU oracle legs
def oracle_pass(cfg, heads, n_tokens):
    """The oracle's whole path for the given KV heads of sample 0: subspace from the n_tokens prompt queries, then
    keys, values and both dequantizers on the prompt's tokens -- or, for the decode-append workload, on the tokens of
    its windows (quantizing them in one call equals window by window: groups never straddle a window).  Yields
    (seconds, key vectors processed)."""
    import oracle
    n_quant = cfg.decode_windows * cfg.decode_window_len if cfg.decode_windows else n_tokens
    for h in heads:
        qs = [si.to_f32(si.gen_queries_head(cfg, hq, n_tokens), cfg.dtype)
              for hq in range(h * cfg.q_per_kv, (h + 1) * cfg.q_per_kv)]
        Qc = np.concatenate(qs, 0).astype(np.float64)
        K = si.to_f32(si.gen_keys_unit(cfg, 0, h, n_quant, 1 if cfg.decode_windows else 0), cfg.dtype)
        V = si.to_f32(si.gen_values_unit(cfg, 0, h, n_quant, 1 if cfg.decode_windows else 0), cfg.dtype)
        t0 = time.perf_counter()
        mats = oracle.build_W(Qc, cfg.rank_r, cfg.lam, cfg.block_g)
        ok = oracle.quant_keys(K.astype(np.float64), cfg.group_size, cfg.bits, mats["W"])
        ov = oracle.quant_values_f32(V, cfg.group_size, cfg.bits)
        oracle.dequant_keys(ok["codes"], ok["scale"], ok["zero"], cfg.group_size)
        oracle.dequant_values(ov["codes"], ov["scale"], ov["zero"], cfg.group_size)
        yield time.perf_counter() - t0, n_quant


def cpu_baseline(cfg, budget_s=12.0):
    """Times the oracle (as it stands, 1 thread) on a bounded sample: as many KV heads of sample 0 as fit
    in the budget (at least one)."""
    import oracle
    oracle.build()
    spent, vecs, heads = 0.0, 0, 0
    for dt, n in oracle_pass(cfg, range(cfg.n_kv_heads), cfg.n_tokens):
        spent += dt; vecs += n; heads += 1
        if spent > budget_s:
            break
    return {"value": vecs / spent, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{heads} of {cfg.n_kv_heads} KV heads of sample 0 of {cfg.name} (all {vecs // heads} quantized tokens each): "
                      f"subspace build + keys + values + dequantize, {spent:.1f} s of CPU time"}


def run_reference(args, cfg):
    rank, _, world = dist_env()
    if rank != 0:
        return
    import oracle
    oracle.build()
    heads_per_step = 2
    times = []
    it = 0
    for step in range(args.warmup + args.steps):
        heads = [(it + i) % cfg.n_kv_heads for i in range(heads_per_step)]
        it += heads_per_step
        dt = sum(t for t, _ in oracle_pass(cfg, heads, cfg.n_tokens))
        if step >= args.warmup:
            times.append(dt)
    vec_per_step = heads_per_step * (cfg.decode_windows * cfg.decode_window_len if cfg.decode_windows else cfg.n_tokens)
    total = sum(times)
    value = vec_per_step * len(times) / total
    sample = (f"each step = {heads_per_step} KV heads of sample 0 of {cfg.name}, all {vec_per_step // heads_per_step} quantized tokens: "
              "subspace build + keys + values + dequantize")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / len(times),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": dict(workload_config(cfg), metadata="float32", subspace="svd"), "gpu_launches": 0,
            "cpu_baseline": {"value": value, "unit": UNIT, "kind": "oracle", "cores": 1, "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def rank_is_zero():
    return dist_env()[0] == 0


def workload_config(cfg):
    return {"workload": f"config {cfg.index}: {cfg.name}", "dtype": cfg.dtype, "batch": cfg.batch,
            "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
            "n_tokens": cfg.n_tokens, "rank_r": cfg.rank_r, "bits": cfg.bits, "group_size": cfg.group_size,
            "lambda": cfg.lam, "block_g": cfg.block_g, "l2": "flushed between steps (512 MiB write)",
            "decode_windows": cfg.decode_windows, "decode_window_len": cfg.decode_window_len,
            "step": ("build from the prompt + %d window calls of keys and of values into a %d-token cache + dequantize of that cache"
                     % (cfg.decode_windows, cfg.decode_windows * cfg.decode_window_len)) if cfg.decode_windows
                    else "build + keys + values + dequantize of one prompt pass",
            "parallelism": "independent replicas per GPU (no collective on the data path)"}


# --------------------------------------------------------------------------- the GPU arm
def run_gpu(args, cfg):
    import torch
    import torch.distributed as dist
    import paper_2503_24358_b200 as sq

    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the write path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group(backend="nccl", device_id=dev)

    def to_dev(a, pin=False):
        if cfg.dtype == "f32":
            t = torch.from_numpy(np.ascontiguousarray(a))
        else:
            t = torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).view(torch.bfloat16)
        return t.pin_memory() if pin else t.to(dev)

    B, H, d, bits, G = cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.bits, cfg.group_size
    stream_mode = cfg.decode_windows > 0
    # prompt pass: one call of each quantizer on the T prompt tokens; decode-append stream: NW calls on W tokens each,
    # written side by side into a cache of Tc = NW * W tokens
    NW = cfg.decode_windows if stream_mode else 1
    W = cfg.decode_window_len if stream_mode else cfg.n_tokens
    Tc = NW * W
    NDIST = min(NW, 8)                        # distinct window tensors, cycled (8 x 128 MiB of k and v: far beyond L2)
    tdt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    q_np = si.gen_queries(cfg)
    if stream_mode:
        k_np = [si.gen_keys(cfg, n_tokens=W, segment=1 + i) for i in range(NDIST)]
        v_np = [si.gen_values(cfg, n_tokens=W, segment=1 + i) for i in range(NDIST)]
    else:
        k_np, v_np = [si.gen_keys(cfg)], [si.gen_values(cfg)]
    q = to_dev(q_np)
    k_w, v_w = [to_dev(a) for a in k_np], [to_dev(a) for a in v_np]
    kc = torch.empty((B, H, Tc, d * bits // 8), dtype=torch.uint8, device=dev)
    mdt = torch.float16 if args.meta16 else torch.float32   # storage type of scales and zero-points
    ks = torch.empty((B, H, Tc // G, d), dtype=mdt, device=dev)
    kz = torch.empty_like(ks)
    vc = torch.empty_like(kc)
    vs = torch.empty((B, H, Tc, d // G), dtype=mdt, device=dev)
    vz = torch.empty_like(vs)
    kd = torch.empty((B, H, Tc, d), dtype=tdt, device=dev)
    vd = torch.empty_like(kd)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    s = sq.Subspace(H, d)
    stream = torch.cuda.current_stream()

    stage_names = ["build_subspace", "quantize_keys", "quantize_values", "dequantize"]
    n_events = 3 + 2 * NW                      # start | build done | (keys, values) per window | dequantize done

    # start block of the block power method (the random numbers that variant draws), resident like the other inputs
    x0 = torch.from_numpy(si.gen_start_block(cfg.seed, d, cfg.rank_r)).to(dev) if 0 < cfg.rank_r <= 64 else None
    use_power = args.subspace == "power"
    if use_power and x0 is None:
        raise SystemExit("--subspace power needs 0 < rank <= 64")

    def build():
        if use_power:
            sq.squat_build_subspace_power(s, q, cfg.rank_r, cfg.lam, x0, args.power_iters, cfg.block_g)
        else:
            sq.squat_build_subspace(s, q, cfg.rank_r, cfg.lam, cfg.block_g)

    def step(ev=None):
        if ev: ev[0].record(stream)
        build()
        if ev: ev[1].record(stream)
        for w in range(NW):
            lo = w * W
            sq.squat_quantize_keys(s, k_w[w % NDIST], bits, G, kc[:, :, lo:], ks[:, :, lo // G:], kz[:, :, lo // G:],
                                   out_stride_b=H * Tc, out_stride_h=Tc)
            if ev: ev[2 + 2 * w].record(stream)
            sq.squat_quantize_values(v_w[w % NDIST], bits, G, vc[:, :, lo:], vs[:, :, lo:], vz[:, :, lo:],
                                     out_stride_b=H * Tc, out_stride_h=Tc)
            if ev: ev[3 + 2 * w].record(stream)
        sq.squat_dequantize(sq.SQUAT_KEYS, kc, ks, kz, B, H, Tc, d, bits, G, kd)
        sq.squat_dequantize(sq.SQUAT_VALUES, vc, vs, vz, B, H, Tc, d, bits, G, vd)
        if ev: ev[2 + 2 * NW].record(stream)

    sq.squat_subspace_select_key_kernel(s, args.dense_keys)
    fp32_peak = measure_fp32_peak(sq, dev) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        flush.zero_()
        step()
    torch.cuda.synchronize()

    props = torch.cuda.get_device_properties(local_rank)
    bus = None
    if all(hasattr(props, a) for a in ("pci_domain_id", "pci_bus_id", "pci_device_id")):
        bus = "%08x:%02x:%02x.0" % (props.pci_domain_id, props.pci_bus_id, props.pci_device_id)
    sampler = ClockSampler(local_rank, bus)
    if rank == 0:
        sampler.start()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    launches0 = sq.squat_kernel_launch_count()
    events = [[torch.cuda.Event(enable_timing=True) for _ in range(n_events)] for _ in range(args.steps)]
    wall0 = time.perf_counter()
    for i in range(args.steps):
        flush.zero_()                      # evict inputs and outputs from L2 (not part of a step's time)
        step(events[i])
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    wall = time.perf_counter() - wall0
    clocks = sampler.stop() if rank == 0 else None
    if rank == 0 and not clocks.get("samples"):
        # no sample landed inside the (short) timed region: repeat the same loop untimed under a fresh sampler
        sampler = ClockSampler(local_rank, bus)
        sampler.start()
        t_end = time.perf_counter() + 0.5
        while time.perf_counter() < t_end:
            flush.zero_()
            step()
            torch.cuda.synchronize()
        clocks = sampler.stop()
        clocks["sampled"] = "in an untimed repeat of the timed loop right after it (no sample landed inside the timed region)"
    launches = sq.squat_kernel_launch_count() - launches0
    last = 2 + 2 * NW
    step_ms = [e[0].elapsed_time(e[last]) for e in events]
    key_calls = [[e[1 + 2 * w].elapsed_time(e[2 + 2 * w]) for w in range(NW)] for e in events]      # [step][window]
    val_calls = [[e[2 + 2 * w].elapsed_time(e[3 + 2 * w]) for w in range(NW)] for e in events]
    stage_ms = {"build_subspace": statistics.mean(e[0].elapsed_time(e[1]) for e in events),
                "quantize_keys": statistics.mean(sum(c) for c in key_calls),
                "quantize_values": statistics.mean(sum(c) for c in val_calls),
                "dequantize": statistics.mean(e[last - 1].elapsed_time(e[last]) for e in events)}
    stream_stats = None
    if stream_mode:
        seq_ms = [e[1].elapsed_time(e[last - 1]) for e in events]               # the NW (keys, values) pairs, build and read-back excluded
        flat_k = [c for st in key_calls for c in st]
        flat_v = [c for st in val_calls for c in st]
        flat_p = [a + b_ for sk, sv in zip(key_calls, val_calls) for a, b_ in zip(sk, sv)]
        us = lambda xs: {"median_us": 1e3 * statistics.median(xs), "best_us": 1e3 * min(xs), "mean_us": 1e3 * statistics.mean(xs)}
        stream_stats = {
            "what": "%d window calls per step, each squat_quantize_keys + squat_quantize_values on [%d, %d, %d, %d] written at "
                    "its offset of a %d-token cache; the subspace comes from the %d-token prompt" % (NW, B, H, W, d, Tc, cfg.n_tokens),
            "calls_timed": len(flat_k), "keys_call": us(flat_k), "values_call": us(flat_v), "window_pair": us(flat_p),
            "sequence_ms": statistics.mean(seq_ms), "sequence_best_ms": min(seq_ms),
            "sequence_key_vectors_per_s": B * H * Tc / (statistics.mean(seq_ms) * 1e-3),
            "timing": "CUDA events on the launching stream between consecutive calls: launch gaps are inside the intervals",
            "distinct_window_tensors": NDIST}
    lowrank_r = sq.squat_subspace_select_key_kernel(s, args.dense_keys)      # which key kernel the steps ran (0: the dense one)
    if args.dense_keys:
        lowrank_r = 0
    local_ms = sum(step_ms)
    vec_per_step = B * H * Tc              # key vectors one step really quantizes
    total_ms, total_units = aggregate_over_ranks(local_ms, vec_per_step * args.steps, dev)
    flags = sq.squat_get_device_status(clear=True)

    # ---- step 1 with the block power method, timed on its own beside the default (SVD) build ------------
    power = None
    if rank == 0 and x0 is not None and not use_power:
        n_p = max(3, min(args.steps, 20))
        pev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_p)]
        for i in range(-2, n_p):
            flush.zero_()
            if i >= 0: pev[i][0].record(stream)
            sq.squat_build_subspace_power(s, q, cfg.rank_r, cfg.lam, x0, args.power_iters, cfg.block_g)
            if i >= 0: pev[i][1].record(stream)
        torch.cuda.synchronize()
        p_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in pev)
        power = {"ms": p_ms, "iters": args.power_iters, "api": "squat_build_subspace_power",
                 "note": "Gram + block power iteration + update matrices; not part of the timed step "
                         "(run with --subspace power to time the whole path with it)",
                 "whole_path_ms_with_it": statistics.mean(step_ms) - stage_ms["build_subspace"] + p_ms}
        sq.squat_build_subspace(s, q, cfg.rank_r, cfg.lam, cfg.block_g)      # leave the handle as the step left it
        torch.cuda.synchronize()

    # ---- the same step with the value path on a second stream: values and their read-back do not depend on the subspace,
    # so they can run beside build -> keys -> read-back of the keys (the library calls take any stream) -------------
    overlapped = None
    if rank == 0 and not stream_mode:
        side = torch.cuda.Stream()
        n_o = max(3, min(args.steps, 20))
        oev = [[torch.cuda.Event(enable_timing=True) for _ in range(2)] for _ in range(n_o)]
        join = torch.cuda.Event()
        for i in range(-2, n_o):
            flush.zero_()
            if i >= 0: oev[i][0].record(stream)
            side.wait_stream(stream)
            with torch.cuda.stream(side):
                sq.squat_quantize_values(v_w[0], bits, G, vc, vs, vz, stream=side)
                sq.squat_dequantize(sq.SQUAT_VALUES, vc, vs, vz, B, H, Tc, d, bits, G, vd, stream=side)
                join.record(side)
            build()
            sq.squat_quantize_keys(s, k_w[0], bits, G, kc, ks, kz)
            sq.squat_dequantize(sq.SQUAT_KEYS, kc, ks, kz, B, H, Tc, d, bits, G, kd)
            stream.wait_event(join)
            if i >= 0: oev[i][1].record(stream)
        torch.cuda.synchronize()
        o_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in oev)
        overlapped = {"ms_per_step": o_ms, "key_vectors_per_s": vec_per_step / (o_ms * 1e-3),
                      "what": "values + their read-back on a second stream beside build -> keys -> read-back of the keys; "
                              "not the timed step (which issues every call on one stream)"}

    # ---- end to end from host buffers --------------------------------------------------------------
    e2e = None
    if not args.no_e2e:
        if stream_mode:
            e2e = run_e2e_stream(args, cfg, sq, s, q_np, k_np, v_np, to_dev, flush, tdt, mdt, dev, vec_per_step, NW, W, NDIST)
        else:
            e2e = run_e2e(args, cfg, sq, s, (q_np, k_np[0], v_np[0]), (kc, ks, kz, vc, vs, vz), to_dev, flush, tdt, dev,
                          vec_per_step)
    # ---- the reader that follows the write path (not part of a step): one decode step of attention -----
    reader = None
    if rank == 0 and not args.no_reader:
        reader = run_reader(cfg, sq, (kc, ks, kz, vc, vs, vz), Tc, flush, tdt, dev, meta_bytes=2 if args.meta16 else 4)
    if rank == 0:
        key_launch_ms = stage_ms["quantize_keys"] / NW
        report(args, cfg, world, total_ms, total_units, step_ms, stage_ms, stage_names, vec_per_step, B * H * W, key_launch_ms,
               e2e, launches, wall, flags, clocks, fp32_peak, reader, power, stream_stats, lowrank_r, overlapped)
    s.close()
    if world > 1:
        dist.destroy_process_group()


def run_e2e(args, cfg, sq, s, host_np, dev_outs, to_dev, flush, tdt, dev, vec_per_step):
    import torch
    B, H, T, d, bits, G = cfg.batch, cfg.n_kv_heads, cfg.n_tokens, cfg.head_dim, cfg.bits, cfg.group_size
    q_np, k_np, v_np = host_np
    kc, ks, kz, vc, vs, vz = dev_outs
    qh, kh, vh = to_dev(q_np, pin=True), to_dev(k_np, pin=True), to_dev(v_np, pin=True)
    outs_h = [torch.empty_like(t, device="cpu").pin_memory() for t in (kc, ks, kz, vc, vs, vz)]
    ws = torch.empty(sq.squat_write_path_workspace_bytes(tdt, B, cfg.n_q_heads, H, T, d, bits, G), dtype=torch.uint8,
                     device=dev)
    h2d = sum(t.numel() * t.element_size() for t in (qh, kh, vh))
    d2h = sum(t.numel() * t.element_size() for t in outs_h)
    e2e_steps = max(3, min(args.steps, 10))
    # the same entry serves the variants: float16 metadata tensors -> 16-bit cache; a start block -> block power build
    x0h = None
    if args.subspace == "power":
        x0h = torch.from_numpy(si.gen_start_block(cfg.seed, d, cfg.rank_r)).pin_memory()
    kw = {"start_block": x0h, "power_iters": args.power_iters}
    for _ in range(2):
        sq.squat_write_path_host(s, qh, kh, vh, cfg.rank_r, cfg.lam, cfg.block_g, bits, G, *outs_h, ws, **kw)
    e2e_ms = []
    for _ in range(e2e_steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        sq.squat_write_path_host(s, qh, kh, vh, cfg.rank_r, cfg.lam, cfg.block_g, bits, G, *outs_h, ws, **kw)
        e2e_ms.append(1e3 * (time.perf_counter() - t0))        # the call synchronises its stream
    e2e_total_ms, e2e_units = aggregate_over_ranks(sum(e2e_ms), vec_per_step * e2e_steps, dev)
    return {"value": e2e_units / (e2e_total_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": e2e_total_ms / e2e_steps,
            "api": "squat_write_path_host%s (pinned host buffers; build + keys + values)"
                   % ("_ex" if (args.meta16 or args.subspace == "power") else "")}


def run_e2e_stream(args, cfg, sq, s, q_np, k_np, v_np, to_dev, flush, tdt, mdt, dev, vec_per_step, NW, W, NDIST):
    """The decode-append stream from pinned host buffers: the prompt's queries go up and the subspace is built, then
    every window goes through squat_append_window_host (its keys and values up, both quantizers, its codes, scales and
    zero-points down).  Wall-clock around the whole sequence; every call synchronises its stream."""
    import torch
    B, H, d, bits, G = cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.bits, cfg.group_size
    qh = to_dev(q_np, pin=True)
    q_dev = torch.empty_like(qh, device=dev)
    kh = [to_dev(a, pin=True) for a in k_np]
    vh = [to_dev(a, pin=True) for a in v_np]
    outs_h = [torch.empty(shape, dtype=dt).pin_memory() for shape, dt in (
        ((B, H, W, d * bits // 8), torch.uint8), ((B, H, W // G, d), mdt), ((B, H, W // G, d), mdt),
        ((B, H, W, d * bits // 8), torch.uint8), ((B, H, W, d // G), mdt), ((B, H, W, d // G), mdt))]
    ws = torch.empty(sq.squat_write_path_workspace_bytes(tdt, B, H, H, W, d, bits, G), dtype=torch.uint8, device=dev)
    h2d = qh.numel() * qh.element_size() + NW * 2 * kh[0].numel() * kh[0].element_size()
    d2h = NW * sum(t.numel() * t.element_size() for t in outs_h)
    e2e_steps = max(3, min(args.steps, 5))

    def one_step(call_ms=None):
        q_dev.copy_(qh, non_blocking=True)
        sq.squat_build_subspace(s, q_dev, cfg.rank_r, cfg.lam, cfg.block_g)
        for w in range(NW):
            t0 = time.perf_counter()
            sq.squat_append_window_host(s, kh[w % NDIST], vh[w % NDIST], bits, G, *outs_h, ws)
            if call_ms is not None:
                call_ms.append(1e3 * (time.perf_counter() - t0))

    one_step()
    e2e_ms, call_ms = [], []
    for _ in range(e2e_steps):
        flush.zero_()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        one_step(call_ms)
        torch.cuda.synchronize()
        e2e_ms.append(1e3 * (time.perf_counter() - t0))
    e2e_total_ms, e2e_units = aggregate_over_ranks(sum(e2e_ms), vec_per_step * e2e_steps, dev)
    return {"value": e2e_units / (e2e_total_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
            "d2h_bytes_per_step": d2h, "ms_per_step": e2e_total_ms / e2e_steps,
            "window_call_ms": {"median": statistics.median(call_ms), "best": min(call_ms)},
            "api": "host->device copy of the prompt queries + squat_build_subspace, then %d x squat_append_window_host "
                   "(pinned host buffers; keys + values of one window up, quantized, outputs down)" % NW}


def run_reader(cfg, sq, cache, T, flush, tdt, dev, iters=10, meta_bytes=4):
    """One decode step of attention over the cache the step has just written (plus a full residual buffer of
    random full-precision rows): time per call and the bytes it has to read, against the copy bandwidth."""
    import torch
    B, H, d, bits, G = cfg.batch, cfg.n_kv_heads, cfg.head_dim, cfg.bits, cfg.group_size
    Hq, R = cfg.n_q_heads, (cfg.residual or 32)
    gen = torch.Generator(device=dev).manual_seed(1234)
    q = torch.randn(B, Hq, d, generator=gen, device=dev).to(tdt)
    k_res = torch.randn(B, H, R, d, generator=gen, device=dev).to(tdt)
    v_res = torch.randn(B, H, R, d, generator=gen, device=dev).to(tdt)
    out = torch.empty((B, Hq, d), dtype=torch.float32, device=dev)
    ws = torch.empty(sq.squat_decode_attention_workspace_bytes(B, Hq, T), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    def timed(call):
        for _ in range(3):
            flush.zero_()
            call()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(iters)]
        for a, b in ev:
            flush.zero_()
            a.record(stream)
            call()
            b.record(stream)
        torch.cuda.synchronize()
        return statistics.mean(a.elapsed_time(b) for a, b in ev)

    ms = timed(lambda: sq.squat_decode_attention(q, *cache, H, T, bits, G, out, ws, k_res, v_res))
    # the same step when the keys were stored before the rotary embedding (the cache's bytes are read as un-rotated
    # keys at positions 0 .. T + R - 1; timing only, the parity tests cover the arithmetic)
    table = sq.squat_rope_table(T + R).to(dev)
    ms_pre = timed(lambda: sq.squat_decode_attention_pre_rope(q, *cache, H, T, bits, G, out, ws, table, T + R, 0, k_res, v_res))
    elem = 4 if cfg.dtype == "f32" else 2
    toks = B * H * T
    nbytes = toks * reader_bytes_per_cached_token(d, bits, G, meta_bytes) + 2 * B * H * R * d * elem + B * Hq * d * (elem + 4)
    peaks = measured_peaks()
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"what": "squat_decode_attention: softmax(q K^T / sqrt(d)) V over the packed cache + residual buffer",
            "ms_per_call": ms, "cached_tokens": toks, "n_q_heads": Hq, "residual_tokens": R, "bytes_per_call": nbytes,
            "hbm_gbs": gbs, "hbm_frac": gbs / peaks["hbm_gbs"], "cached_tokens_per_s": toks / (ms * 1e-3),
            "pre_rope": {"what": "squat_decode_attention_pre_rope: the same step with the rotary embedding applied to "
                                 "the dequantized keys on the fly", "ms_per_call": ms_pre,
                         "hbm_gbs": nbytes / (ms_pre * 1e-3) / 1e9, "hbm_frac": nbytes / (ms_pre * 1e-3) / 1e9 / peaks["hbm_gbs"],
                         "slowdown": ms_pre / ms}}


def key_roofline(args, cfg, key_ms, vec_per_launch, peaks, fp32_peak, lowrank_r=0):
    """The roofline of the key kernel: the slowest of (the multiply-adds it runs on the FP32 pipes at the FP32 peak
    measured in this run, three tf32 products per cross-block multiply-add at the tf32 peak, the bytes at the measured
    HBM copy bandwidth) against the measured time of one launch.  `frac` = achieved / peak on the pipe that sets that
    floor.  The figure the 50 % target was first stated in -- every algorithmic flop at the nominal FP32 peak -- is kept
    as frac_vs_fp32_target."""
    d, bits, G = cfg.head_dim, cfg.bits, cfg.group_size
    elem = 4 if cfg.dtype == "f32" else 2
    mb = 2 if args.meta16 else 4
    t_s = key_ms * 1e-3
    alg_flops = key_flops_per_vector(d, cfg.block_g, cfg.rank_r) * vec_per_launch
    kbytes = bytes_per_vector(d, bits, G, elem, mb) * vec_per_launch
    alu_fma, tensor_fma = key_fma_split(d, cfg.block_g)
    if lowrank_r > 0:
        alu_fma, tensor_fma = 2 * lowrank_r * d, 0                # the rank-r form: state of r numbers per token, FP32 pipes only
    if cfg.rank_r == 0 or cfg.lam == 0.0:
        alu_fma = tensor_fma = 0                                  # W = 0: nothing to push
    fp32_tflops = fp32_peak["tflops"] if fp32_peak else ALU_PEAK_TFLOPS
    tf32_peak = 0.5 * peaks["bf16_tflops"]                        # nominal ratio tf32 : bf16 = 1 : 2
    work = {"alu": (2 * alu_fma * vec_per_launch / 1e12, fp32_tflops, "TFLOP/s"),
            "tensor": (3 * 2 * tensor_fma * vec_per_launch / 1e12, tf32_peak, "TFLOP/s"),
            "hbm": (kbytes / 1e9, peaks["hbm_gbs"], "GB/s")}
    floors_us = {k: w / p * 1e6 for k, (w, p, _) in work.items()}
    bound = max(floors_us, key=floors_us.get)
    w, p, unit = work[bound]
    roof = {"bound": bound, "achieved": w / t_s, "peak": p, "unit": unit, "frac": (w / t_s) / p,
            "peak_source": {"alu": "measured in this run: FP32 multiply-add probe kernel (squat_fp32_peak_probe)" if fp32_peak
                                   else "nominal", "tensor": "%s bf16 GEMM peak x 1/2 (nominal tf32 : bf16)" % peaks["source"],
                            "hbm": peaks["source"] + " copy bandwidth"}[bound],
            "definition": "slowest of the three floors below / measured launch time; achieved and peak are those of the "
                          "pipe that sets the floor",
            "pipes": {"fp32_fma_per_vector": alu_fma, "tensor_fma_per_vector": tensor_fma, "tf32_products_per_fma": 3,
                      "fp32_peak_tflops": fp32_tflops, "fp32_peak_measured": fp32_peak, "fp32_peak_nominal_tflops": ALU_PEAK_TFLOPS,
                      "tf32_peak_tflops": tf32_peak, "hbm_peak_gbs": peaks["hbm_gbs"],
                      "fp32_floor_us": floors_us["alu"], "tensor_floor_us": floors_us["tensor"], "hbm_floor_us": floors_us["hbm"],
                      "floor_us": floors_us[bound]},
            "frac_vs_fp32_target": alg_flops / t_s / 1e12 / ALU_PEAK_TFLOPS,
            "frac_vs_fp32_target_definition": "all %d algorithmic flop per vector (2 x min(dense triangle, 2 r d)) at the nominal "
                                              "FP32 peak of %.2f TFLOP/s: the reading the 50 %% target was stated in"
                                              % (key_flops_per_vector(d, cfg.block_g, cfg.rank_r), ALU_PEAK_TFLOPS),
            "traffic": None, "kernel": "quant_keys_lowrank_kernel (rank-r form of the update)" if lowrank_r > 0 else "quant_keys_kernel", "ms_per_launch": key_ms, "key_vectors_per_launch": vec_per_launch,
            "key_vectors_per_s": vec_per_launch / t_s, "kv_input_gbs": vec_per_launch * d * elem / t_s / 1e9,
            "hbm_frac_of_" + peaks["source"]: kbytes / t_s / 1e9 / peaks["hbm_gbs"]}
    tr = key_kernel_traffic(cfg, args)
    if tr:
        roof["traffic"] = tr["dram_bytes_per_launch"]
        roof["traffic_source"] = tr
        roof["traffic_over_algorithmic_bytes"] = tr["dram_bytes_per_launch"] / kbytes
    return roof


def report(args, cfg, world, total_ms, total_units, step_ms, stage_ms, stage_names, vec_per_step, vec_per_launch, key_launch_ms,
           e2e, launches, wall, flags, clocks, fp32_peak, reader=None, power=None, stream_stats=None, lowrank_r=0, overlapped=None):
    d, bits, G = cfg.head_dim, cfg.bits, cfg.group_size
    if rank_is_zero():
        peaks = measured_peaks()
        elem = 4 if cfg.dtype == "f32" else 2
        mb = 2 if args.meta16 else 4
        roof = key_roofline(args, cfg, key_launch_ms, vec_per_launch, peaks, fp32_peak, lowrank_r)
        # the HBM-bound stages, for the record
        vbytes = bytes_per_vector(d, bits, G, elem, mb) * vec_per_step
        dq_bytes = 2 * (d * bits // 8 + 2 * mb * d // G + d * elem) * vec_per_step
        stages = {n: {"ms": stage_ms[n], "share": stage_ms[n] / statistics.mean(step_ms)} for n in stage_names}
        stages["quantize_values"]["hbm_gbs"] = vbytes / (stage_ms["quantize_values"] * 1e-3) / 1e9
        stages["quantize_values"]["hbm_frac"] = stages["quantize_values"]["hbm_gbs"] / peaks["hbm_gbs"]
        stages["dequantize"]["hbm_gbs"] = dq_bytes / (stage_ms["dequantize"] * 1e-3) / 1e9
        stages["dequantize"]["hbm_frac"] = stages["dequantize"]["hbm_gbs"] / peaks["hbm_gbs"]
        stages["build_subspace"]["method"] = ("block power, %d multiplications" % args.power_iters
                                              if args.subspace == "power" else "svd (fp64 eigen-decomposition)")
        if power is not None:
            stages["build_subspace"]["block_power_variant"] = power
        line = {
            "metric": METRIC, "value": total_units / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
            "config": dict(workload_config(cfg), metadata="binary16" if args.meta16 else "float32",
                           subspace=args.subspace),
            "kv_ingested_gbs": 2 * vec_per_step * world * d * elem / (total_ms / args.steps * 1e-3) / 1e9,
            "roofline": roof, "stages": stages,
            "e2e": e2e,
            "gpu_launches": int(launches), "wall_s_timed_region": wall, "device_status_flags": int(flags),
            "clocks": clocks,
            "cpu_baseline": cpu_baseline(cfg) if (world == 1 and not args.no_cpu_baseline) else None,
            "reader_decode_attention": reader,
        }
        if stream_stats is not None:
            line["decode_append_stream"] = stream_stats
        if overlapped is not None:
            line["overlapped_step"] = overlapped
        print(json.dumps(line))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--no-reader", action="store_true", help="skip the decode-attention leg that follows the step")
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=1, help="workload index (default 1: Llama-2-7B-shaped layer)")
    ap.add_argument("--bits", type=int, default=None, choices=[2, 4], help="override the workload's code width")
    ap.add_argument("--rank", type=int, default=None, help="override the workload's subspace rank r")
    ap.add_argument("--group-size", type=int, default=None, choices=[32, 64, 128], help="override the workload's group size G")
    ap.add_argument("--meta16", action="store_true", help="store scales and zero-points as binary16 (the 18.75 %% cache); "
                    "times the write path only")
    ap.add_argument("--subspace", default="svd", choices=["svd", "power"], help="step 1: the paper's SVD (default) or the "
                    "block power method it names as an accelerator")
    ap.add_argument("--power-iters", type=int, default=2, help="multiplications by the Gram matrix of the block power method")
    ap.add_argument("--dense-keys", action="store_true", help="run the dense key kernel also where the rank-r form of the "
                    "update is available (small ranks)")
    ap.add_argument("--impl", default="squat", choices=["squat", "reference"])
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    ap.add_argument("--no-cpu-baseline", action="store_true", help="skip the oracle timing (profiling runs)")
    args = ap.parse_args()
    cfg = si.get_config(args.config)
    over = {k: v for k, v in (("bits", args.bits), ("rank_r", args.rank), ("group_size", args.group_size)) if v is not None}
    if over:                                             # one point of a workload's (bits, r, G) sweep
        cfg = cfg.with_(**over)
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_gpu(args, cfg)


if __name__ == "__main__":
    main()

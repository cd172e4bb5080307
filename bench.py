#!/usr/bin/env python
"""Benchmark of the streaming decoder step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg5|cfg3|cfg2|cfg4|cfg1]
    python bench.py --impl reference ...        # the CPU oracle, timed on the host cores

A step is one pass of the whole per-chunk hot path over one batch of synthetic input: for the
multi-stream workload (default, cfg5) one dc_decode_batch call that advances each of the 32
streams by one 50-frame chunk (= 1 s of audio per stream); for the single-stream workloads one
dc_decode_chunk call.  Prints ONE JSON line on rank 0.

Multi-GPU: the path does not shard (a stream is strictly sequential), so --gpus N runs N
independent replicas, one process per GPU, each with its own streams ("replicas only"); the only
cross-rank traffic is the barrier and the max-over-ranks of the timing.
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
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import dc_workloads as wl  # noqa: E402

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# FP32 FFMA peak of the part as derived from its unit counts: 148 SMs x 128 lanes x 2 flop x 1.965 GHz; the bench
# divides by the figure it MEASURES in the run (dc_measure_fp32_peak) and prints the derived one beside it
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
HISTORY_CHUNKS = 12      # untimed stream history so that the K/V carry sits at its cap (steady state)
# dram__bytes_read.sum + dram__bytes_write.sum per launch of the dominant kernel, from an ncu capture of
# this command (a figure of a capture, not read in the run; None until a capture exists for that workload)
NCU_TRAFFIC_BYTES = {"cfg5": 4.00e6,   # conv-mode flow_gemm_kernel
                     "cfg3": None, "cfg2": None, "cfg4": None, "cfg1": None}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS if k in d}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []      # (host time of arrival, fields)
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) >= 7:
                self.rows.append((time.perf_counter(), parts))

    def stop(self, windows=None):
        """windows: {name: (t0, t1)} host-time intervals; the summary uses the samples that arrived
        inside any of them (a sample describes the ~50 ms before its arrival) and counts them per window."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        counts = {}
        rows = []
        for t, parts in self.rows:
            for name, (t0, t1) in (windows or {"all": (0.0, float("inf"))}).items():
                if t0 <= t <= t1 + 0.06:
                    counts[name] = counts.get(name, 0) + 1
                    rows.append(parts)
                    break
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        pw = [float(r[2]) for r in rows if r[2].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[3 + i] == "Active" for r in rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": statistics.median(pw) if pw else None, "reasons": reasons, "samples": len(rows),
                "samples_by_window": counts, "period_ms": 50}


def describe(cfg) -> str:
    if cfg.pipeline == "token2wav":
        return (describe(cfg.flow_part()).replace(cfg.name + ".flow", cfg.name) + " -> mel frames on the device -> "
                + describe(cfg.vocoder_part()).split(": ", 1)[1])
    if cfg.pipeline == "flow":
        return (f"{cfg.name}: {cfg.n_streams} stream(s) x flow decoder C={cfg.hidden}, {len(cfg.dilations)} conv blocks, "
                f"{cfg.n_attn_layers} attention layers ({cfg.n_heads}x{cfg.head_dim}, KV cap {cfg.kv_cap}), "
                f"{cfg.n_steps} Euler steps, {cfg.f_chunk}-frame chunks, bf16 / fp32 accumulate"
                + (f", classifier-free guidance w={cfg.cfg_scale} (two passes per step)" if cfg.cfg_scale > 0 else "")
                + (f", {cfg.f_prompt}-frame prompt kept in the carry" if cfg.f_prompt > 0 else "")
                + (f", {cfg.f_lookahead} look-ahead frames per call" if cfg.f_lookahead > 0 else ""))
    if cfg.pipeline == "vocoder":
        return (f"{cfg.name}: vocoder tail mel {cfg.mel_dim} -> strides {cfg.up_strides} channels {cfg.up_channels} "
                f"-> head -> iSTFT n_fft {cfg.n_fft} hop {cfg.hop}, {cfg.f_chunk}-frame chunks, fp32")
    return f"{cfg.name}: causal conv stream C={cfg.hidden} dilations {cfg.dilations}, {cfg.f_chunk}-frame chunks, fp32"


def units_per_chunk(cfg):
    """(metric, unit, units one chunk of one stream is worth)."""
    if cfg.pipeline == "conv":
        return "streamed_frames_per_second", "frames/s", float(cfg.f_chunk)
    return "streamed_audio_seconds_per_second", "audio-s/s", cfg.f_chunk / 50.0   # 50 frames = 1 s of 24 kHz audio


def flops_per_launch(cfg, cls: str, n_streams: int) -> float:
    """Algorithmic FLOPs of one launch of a kernel class (valid rows only)."""
    rows = n_streams * cfg.f_chunk * (2 if getattr(cfg, "cfg_scale", 0.0) > 0 else 1)   # guidance: two passes per stream
    C = cfg.hidden
    if cls == "gemm_conv":
        return 2.0 * rows * C * 3 * C
    if cls == "attention":
        L = getattr(cfg, "f_prompt", 0) + cfg.kv_cap + cfg.f_chunk
        return 2.0 * 2.0 * rows * L * C
    return 0.0


def flow_step_work(cfg, n_streams: int):
    """Algorithmic FLOPs and HBM bytes of one whole chunk step of a flow decoder (all Euler steps, valid rows)."""
    rows = n_streams * cfg.f_chunk * (2 if getattr(cfg, "cfg_scale", 0.0) > 0 else 1)
    C, mel = cfg.hidden, cfg.mel_dim
    n_conv, n_attn = len(cfg.dilations), cfg.n_attn_layers
    per_step = (2.0 * rows * 2 * mel * C                       # input projection
                + n_conv * 2.0 * rows * C * 3 * C              # conv blocks
                + n_attn * (2.0 * rows * C * 3 * C             # QKV projection
                            + flops_per_launch(cfg, "attention", n_streams)
                            + 2.0 * rows * C * C)              # attention output projection
                + 2.0 * rows * C * mel)                        # output projection
    by = cfg.n_steps * n_attn * attention_bytes_per_launch(cfg, n_streams)   # the K/V sweeps; weights and activations live in L2
    return cfg.n_steps * per_step, by


def attention_bytes_per_launch(cfg, n_streams: int) -> float:
    """K and V rows of the attended window (bf16) + Q read + O write."""
    L = getattr(cfg, "f_prompt", 0) + cfg.kv_cap + cfg.f_chunk + getattr(cfg, "f_lookahead", 0)
    passes = 2 if getattr(cfg, "cfg_scale", 0.0) > 0 else 1
    return passes * n_streams * (2.0 * L * cfg.hidden * 2 + 2.0 * cfg.f_chunk * cfg.hidden * 2)


def max_over_ranks(value: float, world: int, device: str = "cuda") -> float:
    """Max of a per-rank scalar over all ranks (the replicas only meet here and at the barrier)."""
    if world <= 1:
        return value
    import torch
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_throughput(world: int, streams_per_rank: int, steps: int, per_chunk: float, seconds: float) -> float:
    """Whole-job units per second: every rank advances its own streams by `steps` chunks (weak scaling)."""
    return world * streams_per_rank * steps * per_chunk / seconds


def cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def time_oracle(cfg, weights, feats, budget_s: float = 12.0, min_chunks: int = 8, max_chunks: int = 4000):
    """Times the oracle as it stands on consecutive chunks of one stream until about budget_s
    seconds of CPU work are done (the available input chunks are reused cyclically: their values
    do not change the work).  Returns (chunks, seconds)."""
    from oracle import dc_oracle as orc
    st = orc.make_stream(cfg, weights)
    avail = feats.shape[0] // cfg.f_chunk
    t0 = time.perf_counter()
    n = 0
    while n < max_chunks and (n < min_chunks or time.perf_counter() - t0 < budget_s):
        c = n % avail
        st.decode_chunk(feats[c * cfg.f_chunk:(c + 1) * cfg.f_chunk])
        n += 1
    return n, time.perf_counter() - t0


def run_reference(args, cfg):
    """--impl reference: the CPU oracle, one chunk of one stream per step."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import dc_oracle as orc
    metric, unit, per_chunk = units_per_chunk(cfg)
    rng = np.random.default_rng(cfg.seed)
    weights = wl.make_weights(cfg, rng)
    total = args.warmup + args.steps
    feats = rng.standard_normal((total * cfg.f_chunk, cfg.in_dim), dtype=np.float32)
    st = orc.make_stream(cfg, weights)
    for c in range(args.warmup):
        st.decode_chunk(feats[c * cfg.f_chunk:(c + 1) * cfg.f_chunk])
    t0 = time.perf_counter()
    for c in range(args.warmup, total):
        st.decode_chunk(feats[c * cfg.f_chunk:(c + 1) * cfg.f_chunk])
    dt = time.perf_counter() - t0
    value = per_chunk * args.steps / dt
    cores = cpu_threads()
    sample = f"one chunk of one stream per step ({args.steps} steps after {args.warmup} warm-up chunks, carry growing from empty)"
    print(json.dumps({
        "impl": "reference", "metric": metric, "value": value, "unit": unit, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(cfg), "sample": sample},
        "cpu_baseline": {"value": value, "unit": unit, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": unit, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=60)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg5", choices=sorted(wl.CONFIGS) + sorted(wl.EXTRA_CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--repeats", type=int, default=5,
                    help="runs of history + warm-up + K timed steps, each on freshly opened streams (median reported; 1 for profiler captures)")
    ap.add_argument("--cta-pairs", action="store_true",
                    help="flow decoder: conv and QKV GEMMs of full batches on pairs of SMs (DC_OPT_CTA_PAIRS; same bytes, measured slower)")
    ap.add_argument("--history", type=int, default=None,
                    help="untimed chunks decoded per stream before warm-up (default: enough to fill the K/V carry)")
    args = ap.parse_args()
    cfg = wl.CONFIGS.get(args.workload) or wl.EXTRA_CONFIGS[args.workload]
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import paper_2609_35115_b200 as dc

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the decoder step has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dc.load_library()

    metric, unit, per_chunk = units_per_chunk(cfg)
    S, T = cfg.n_streams, cfg.f_chunk
    Tp = T + getattr(cfg, "f_lookahead", 0)     # frames a call presents; it commits (and is credited with) T
    W, K = max(args.warmup, 3), args.steps
    has_flow = cfg.pipeline in ("flow", "token2wav")
    history = HISTORY_CHUNKS if has_flow else 2
    if args.history is not None:
        history = args.history
    rounds = history + W + K
    rng = np.random.default_rng(cfg.seed + 1000 * rank)
    weights = wl.make_weights(cfg, np.random.default_rng(cfg.seed))
    base_options = dc.OPT_CTA_PAIRS if args.cta_pairs else 0
    model = dc.Model(cfg, weights, max_batch=S, options=base_options)
    feats_h = torch.from_numpy(rng.standard_normal((rounds, S, Tp, cfg.in_dim), dtype=np.float32))
    feats_d = feats_h.cuda()
    out_all = torch.empty(K, S, T * cfg.out_per_frame, device="cuda")     # every timed step's output, hashed after the run
    out_d = out_all[0]
    as_rows = cfg.pipeline not in ("vocoder", "token2wav")
    out_dv = out_d.view(S, T, -1) if as_rows else out_d
    batched = cfg.pipeline in ("flow", "token2wav") and S > 1
    batched_host = batched                              # dc_decode_batch_host: one call per step for all the streams
    # multi-stream serving: the streams' chunk boundaries are staggered by seeded offsets in [0, f_chunk) - stream i's
    # first chunk has o_i frames (a full chunk if o_i = 0), every later one f_chunk
    offsets = np.random.default_rng(cfg.seed).integers(0, T, S) if (batched and S > 1) else np.zeros(S, dtype=np.int64)
    streams = []

    def step(r, out=None):
        o = out_d if out is None else out
        if batched and r == 0 and offsets.any():
            t0 = [int(x) if x > 0 else T for x in offsets]
            dc.decode_batch(model, streams, [feats_d[0, i, :t0[i]] for i in range(S)], [o[i, :t0[i] * cfg.out_per_frame] for i in range(S)])
        elif batched:
            dc.decode_batch(model, streams, feats_d[r], o.view(S, T, -1) if as_rows else o)
        else:
            for i in range(S):
                streams[i].decode_chunk(feats_d[r, i], out=o[i])

    def sync_all():
        torch.cuda.synchronize()
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
            torch.cuda.synchronize()

    def timed_run():
        """Freshly opened streams, history + warm-up, then exactly K timed steps.  Returns per-step events' times,
        the total, the launch count and a hash of every timed step's output."""
        import hashlib
        for s_ in streams:
            s_.close()
        streams[:] = [model.open_stream() for _ in range(S)]
        for r in range(history + W):
            step(r)
        sync_all()
        c0 = model.counters()
        t_host0 = time.perf_counter()
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(K + 1)]
        evs[0].record()
        for k in range(K):
            step(history + W + k, out_all[k])
            evs[k + 1].record()
        torch.cuda.synchronize()
        t_host1 = time.perf_counter()
        c1 = model.counters()
        digest = hashlib.sha256(out_all.cpu().numpy().tobytes()).hexdigest()
        return {"total_ms": evs[0].elapsed_time(evs[K]), "step_ms": sorted(evs[k].elapsed_time(evs[k + 1]) for k in range(K)),
                "launches": int(c1[5] - c0[5]), "graph_launches": int(c1[7] - c0[7]), "hash": digest, "host": (t_host0, t_host1)}

    sampler = ClockSampler(local)
    sampler.start()          # nvidia-smi needs a moment before its first sample: start it ahead of the timed region
    n_rep = max(1, args.repeats)
    runs = [timed_run() for _ in range(n_rep)]
    if len({r_["hash"] for r_ in runs}) != 1:
        raise SystemExit("bench: the outputs of repeated runs differ (the decoder step must be byte-reproducible)")
    runs_sorted = sorted(runs, key=lambda r_: r_["total_ms"])
    med = runs_sorted[n_rep // 2]
    total_ms, step_ms = med["total_ms"], med["step_ms"]
    c_launches, c_graphs = med["launches"], med["graph_launches"]
    # The timed region of a short run is over before nvidia-smi (50 ms period) has sampled it a few
    # times: keep the same steps running, untimed, for about a second and sample that load as well.
    windows = {f"timed_region_{i}": r_["host"] for i, r_ in enumerate(runs)}
    t_p0 = time.perf_counter()
    k = 0
    while time.perf_counter() - t_p0 < 1.0:
        step(history + W + (k % K))
        k += 1
        if k % 8 == 0:
            torch.cuda.synchronize()
    torch.cuda.synchronize()
    windows["same_steps_untimed"] = (t_p0, time.perf_counter())
    clocks = sampler.stop(windows)
    total_ms = max_over_ranks(total_ms, world)
    value = aggregate_throughput(world, S, K, per_chunk, total_ms * 1e-3)
    repeats = {"runs": n_rep, "ms_per_step": [r_["total_ms"] / K for r_ in runs], "reported": "median run",
               "fresh_streams_per_run": True, "outputs_sha256_identical": True, "sha256": med["hash"][:16]}

    # ---- the same step with L2 flushed first (workloads whose working set fits L2 only): a stream paced
    # at its real-time cadence finds its weights and carries in HBM, not in L2 ----
    ws_mb = (S * (cfg.n_steps * cfg.n_attn_layers * 2 * (cfg.f_prompt + cfg.kv_cap + T) * cfg.hidden * 2) / 1e6) if has_flow else 0.0
    cold = None
    if ws_mb <= 126:
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        pairs = []
        for k in range(min(K, 20)):
            flush.fill_(k & 0xFF)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            step(history + W + k)
            e1.record()
            pairs.append((e0, e1))
        torch.cuda.synchronize()
        ct = sorted(a.elapsed_time(b) for a, b in pairs)
        cold = {"p50": 1e3 * ct[len(ct) // 2], "p95": 1e3 * ct[min(len(ct) - 1, int(0.95 * len(ct)))], "steps": len(ct),
                "flush": "256 MiB written before every step"}
        del flush

    # ---- end to end through the host-buffer entry points (H2D + decode + D2H + sync per step) ----
    fin = [feats_h[r].pin_memory() for r in range(history + W, rounds)]
    fout = torch.empty(S, T * cfg.out_per_frame).pin_memory()
    fout_v = fout.view(S, T, -1) if cfg.pipeline not in ("vocoder", "token2wav") else fout
    e2e_warm = min(3, K)
    def e2e_step(k):
        if batched_host:
            dc.decode_batch_host(model, streams, fin[k], fout_v)
        else:
            for i in range(S):
                streams[i].decode_chunk_host(fin[k][i], fout[i])
    for k in range(e2e_warm):
        e2e_step(k)
    sync_all()
    t0 = time.perf_counter()
    for k in range(K):
        e2e_step(k)
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s, world)
    e2e_value = aggregate_throughput(world, S, K, per_chunk, e2e_s)

    # ---- offline decoding of the same single stream as a wavefront (n_steps chunks in flight, one per
    # Euler step; same bytes as the chunk-by-chunk calls): what the step costs when the input is all there ----
    wave = None
    if has_flow and S == 1 and world == 1:
        n_wc = 200
        mw = dc.Model(cfg, weights, max_batch=cfg.n_steps, max_wave_frames=n_wc * T if cfg.pipeline == "token2wav" else 0)
        sw = mw.open_stream()
        fw = torch.from_numpy(rng.standard_normal((n_wc * T, cfg.in_dim), dtype=np.float32)).cuda()
        ow = torch.empty(n_wc * T * cfg.out_per_frame, device="cuda")
        for _ in range(3):
            sw.decode_wavefront(fw, out=ow)
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        cw0 = mw.counters()
        a.record()
        n_calls = 3
        for _ in range(n_calls):
            sw.decode_wavefront(fw, out=ow)
        b.record()
        torch.cuda.synchronize()
        cw1 = mw.counters()
        ms_w = a.elapsed_time(b) / n_calls
        wave = {"value": n_wc * per_chunk / (ms_w * 1e-3), "unit": unit, "ms_per_chunk": ms_w / n_wc,
                "chunks_per_call": n_wc, "chunks_in_flight": cfg.n_steps, "calls_timed": n_calls,
                "gpu_launches_per_call": int(cw1[5] - cw0[5]) // n_calls,
                "note": "dc_decode_wavefront on one stream, input resident in HBM; includes the ramp-up and ramp-down passes"}
        sw.close()
        mw.destroy()
        # ... and of several streams at once (dc_decode_wavefront_batch): every pass carries n_steps chunks of each
        n_pass = 2 if getattr(cfg, "cfg_scale", 0.0) > 0 else 1
        n_ws = min(3, 64 // (cfg.n_steps * n_pass))
        if n_ws >= 2:
            mb = dc.Model(cfg, weights, max_batch=n_ws * cfg.n_steps, max_wave_frames=n_wc * T if cfg.pipeline == "token2wav" else 0)
            sb = [mb.open_stream() for _ in range(n_ws)]
            fb = [torch.from_numpy(rng.standard_normal((n_wc * T, cfg.in_dim), dtype=np.float32)).cuda() for _ in range(n_ws)]
            ob = [torch.empty(n_wc * T * cfg.out_per_frame, device="cuda") for _ in range(n_ws)]
            for _ in range(2):
                dc.decode_wavefront_batch(mb, sb, fb, ob)
            torch.cuda.synchronize()
            a.record()
            for _ in range(n_calls):
                dc.decode_wavefront_batch(mb, sb, fb, ob)
            b.record()
            torch.cuda.synchronize()
            ms_b = a.elapsed_time(b) / n_calls
            wave["batch"] = {"streams": n_ws, "value": n_ws * n_wc * per_chunk / (ms_b * 1e-3), "unit": unit,
                             "ms_per_pass": ms_b / (n_wc + cfg.n_steps - 1), "chunks_per_stream": n_wc}
            for s_ in sb:
                s_.close()
            mb.destroy()

    # ---- per-kernel-class device time (separate profiled pass; events between launches slow the step) ----
    pk, how = peaks()
    # Tensor peak to divide by: the burst figure (a GEMM timed alone at full clock) when this run's SM clock sat at
    # its maximum, the sustained one (seconds of GEMM under the power cap) when it did not; the other is printed beside it.
    at_max = bool(clocks.get("sm_mhz") and clocks.get("sm_max_mhz") and clocks["sm_mhz"] >= 0.97 * clocks["sm_max_mhz"])
    tensor_peak = pk["bf16_tflops"] if at_max else pk["bf16_tflops_sustained"]
    tensor_kind = f"bf16 {'burst (SM clock at max during the run)' if at_max else 'sustained'}, {how}"
    nprof = min(K, 3)
    model.profile_begin(1 << 15)
    for k in range(nprof):
        step(history + W + k)
    ms, nl = model.profile_end()
    tot = sum(ms.values()) or 1.0
    kernels = {k: {"launches_per_step": nl[k] // nprof, "ms_per_step": ms[k] / nprof, "share": ms[k] / tot}
               for k in ms if nl[k]}
    dom = max(kernels, key=lambda k: kernels[k]["ms_per_step"])
    avg_s = 1e-3 * ms[dom] / nl[dom]
    if dom in ("gemm_conv", "gemm_pair"):   # (a paired launch is a conv block or a QKV projection: the same FLOPs)
        fl = flops_per_launch(cfg, "gemm_conv", S)
        roof = {"kernel": "flow_gemm_kernel (conv blocks)" if dom == "gemm_conv" else "flow_gemm_kernel<PAIR> (conv blocks and QKV projections on CTA pairs)", "bound": "tensor", "achieved": fl / avg_s / 1e12,
                "peak": tensor_peak, "unit": "TFLOP/s", "peak_kind": tensor_kind,
                "frac_of_sustained_peak": fl / avg_s / 1e12 / pk["bf16_tflops_sustained"]}
    elif dom == "attention":
        by = attention_bytes_per_launch(cfg, S)
        roof = {"kernel": "flow_attn_kernel", "bound": "hbm", "achieved": by / avg_s / 1e9, "peak": pk["hbm_gbs"],
                "unit": "GB/s", "peak_kind": f"copy bandwidth, {how}"}
    elif dom == "tapconv_f32":
        # per stream-chunk; the token2wav workloads carry cfg4's vocoder tail behind every stream
        fl_chunk = S * (1.73e9 if cfg.pipeline in ("vocoder", "token2wav") else 0.79e6)
        fp32_peak = dc.measure_fp32_peak()
        roof = {"kernel": "tapconv_f32_kernel", "bound": "alu", "achieved": fl_chunk / (1e-3 * ms[dom] / nprof) / 1e12,
                "peak": fp32_peak, "unit": "TFLOP/s", "peak_kind": "FP32 FMA, measured in this run (independent FMA chains on every SM)",
                "peak_derived": FP32_PEAK_TFLOPS, "step_frac": fl_chunk / (1e-3 * total_ms / K) / 1e12 / fp32_peak}
    else:
        roof = {"kernel": dom, "bound": "hbm", "achieved": None, "peak": pk["hbm_gbs"], "unit": "GB/s", "peak_kind": how}
    roof["frac"] = (roof["achieved"] / roof["peak"]) if roof["achieved"] else None
    roof["traffic"] = NCU_TRAFFIC_BYTES.get(cfg.name)
    roof["avg_launch_us"] = 1e6 * avg_s
    if "attention" in kernels and dom != "attention":
        a_s = 1e-3 * ms["attention"] / nl["attention"]
        roof["attention_hbm_gbs"] = attention_bytes_per_launch(cfg, S) / a_s / 1e9
        roof["attention_hbm_frac"] = roof["attention_hbm_gbs"] / pk["hbm_gbs"]

    # ---- cost of the two main kernel classes INSIDE the captured graph (flow workloads, N = 1 only) ----
    # The event-bracketed pass above times direct launches: every bracket adds launch latency and
    # takes away the overlap between consecutive kernels.  What a class costs in the real step is the
    # step time with it minus the step time without it: the library can leave a class out of the
    # graph (a measurement-only option of dc_create; the outputs are then meaningless, the timing
    # of everything else is not).
    if has_flow and world == 1:
        def step_ms_without(bits: int) -> float:
            m2 = dc.Model(cfg, weights, max_batch=S, options=bits | base_options)
            st2 = [m2.open_stream() for _ in range(S)]
            def step2(r):
                if batched:
                    dc.decode_batch(m2, st2, feats_d[r], out_dv)
                else:
                    for i in range(S):
                        st2[i].decode_chunk(feats_d[r, i], out=out_d[i])
            for r in range(history + W):
                step2(r)
            torch.cuda.synchronize()
            n2 = min(K, 30)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for k in range(n2):
                step2(history + W + k)
            b.record()
            torch.cuda.synchronize()
            for s2 in st2:
                s2.close()
            m2.destroy()
            return a.elapsed_time(b) / n2
        full_ms = total_ms / K
        n_conv_l = kernels.get("gemm_conv", {}).get("launches_per_step", 0)
        n_att_l = kernels.get("attention", {}).get("launches_per_step", 0)
        in_graph = {"method": "step time minus the step time of a graph without the class, both over CUDA events"}
        if n_conv_l:
            us = 1e3 * (full_ms - step_ms_without(dc.OPT_SKIP_CONV_GEMM)) / n_conv_l
            in_graph["conv_gemm_us"] = us
            in_graph["conv_gemm_tflops"] = flops_per_launch(cfg, "gemm_conv", S) / (us * 1e-6) / 1e12
            in_graph["conv_gemm_frac"] = in_graph["conv_gemm_tflops"] / tensor_peak
            in_graph["conv_gemm_frac_of_sustained_peak"] = in_graph["conv_gemm_tflops"] / pk["bf16_tflops_sustained"]
        if n_att_l:
            us = 1e3 * (full_ms - step_ms_without(dc.OPT_SKIP_ATTENTION)) / n_att_l
            in_graph["attention_us"] = us
            in_graph["attention_hbm_gbs"] = attention_bytes_per_launch(cfg, S) / (us * 1e-6) / 1e9
            in_graph["attention_hbm_frac"] = in_graph["attention_hbm_gbs"] / pk["hbm_gbs"]
        roof["in_graph"] = in_graph
        # the whole step against the two rooflines (the paper's stage bound, Eq. 1: max of the compute time and
        # the memory time), next to the per-kernel figures above
        fl_step, by_step = flow_step_work(cfg, S)   # (token2wav workloads: the flow decoder's part of the work only)
        t_floor = max(fl_step / (tensor_peak * 1e12), by_step / (pk["hbm_gbs"] * 1e9))
        roof["step"] = {"flops": fl_step, "hbm_bytes": by_step, "floor_us": 1e6 * t_floor,
                        "measured_us": 1e3 * full_ms, "frac": t_floor / (1e-3 * full_ms)}
        # the stage-latency floor: the same graph with kernels that return at once (same nodes, same launch attributes);
        # flow workloads only - the composite's vocoder tail has no such switch
        if cfg.pipeline == "flow":
            empty_ms = step_ms_without(dc.OPT_EMPTY_KERNELS)
            n_nodes = c_launches // K
            roof["t_sync"] = {"empty_step_us": 1e3 * empty_ms, "graph_nodes": n_nodes, "t_sync_us": 1e3 * empty_ms / max(n_nodes, 1),
                              "n_stages_x_t_sync_frac_of_step": empty_ms / full_ms,
                              "method": "the step's graph with GEMM and attention kernels that return at once"}

    # ---- the oracle on the host cores (rank 0, N = 1 only), bounded sample ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        f = feats_h[:, 0].reshape(-1, cfg.in_dim).numpy()
        n_c, dt = time_oracle(cfg, weights, f)
        cpu = {"value": n_c * per_chunk / dt, "unit": unit, "cores": cpu_threads(), "kind": "oracle",
               "sample": f"{n_c} consecutive chunks of one stream (carry growing from empty), {dt:.1f} s"}

    if rank == 0:
        ws = ws_mb
        line = {
            "metric": metric, "value": value, "unit": unit, "n_gpus": world, "steps": K, "warmup": W,
            "ms_per_step": total_ms / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": ("bf16+f32" if cfg.pipeline == "token2wav" else "bf16" if cfg.precision == "bf16" else "f32"), "data": "synthetic",
            "config": {"workload": describe(cfg), "streams_per_gpu": S, "frames_per_chunk": T,
                       "history_chunks": history, "cta_pairs": bool(args.cta_pairs), "parallelism": "replicas only" if world > 1 else "1 gpu",
                       "l2": (f"K/V carries {ws:.0f} MB > 126 MB L2, streamed from HBM every step" if ws > 126 else
                              "working set fits L2: value and latency_us are back-to-back chunks (warm L2), latency_us_cold_l2 flushes L2 before every step"),
                       "inputs": "N(0,1) features, N(0,1/fan_in) weights, seeded"
                                 + ("; stream i's first chunk has a seeded o_i in [0, f_chunk) frames (staggered chunk boundaries)" if offsets.any() else ""),
                       "protocol": f"{n_rep} runs of history + warm-up + K timed steps, each on freshly opened streams; outputs hashed, median run reported"},
            "latency_us": {"p50": 1e3 * step_ms[len(step_ms) // 2], "p95": 1e3 * step_ms[min(len(step_ms) - 1, int(0.95 * len(step_ms)))],
                           "per": "step (one chunk of every stream)"},
            "latency_us_cold_l2": cold,
            "wavefront": wave,
            "e2e": {"value": e2e_value, "unit": unit, "h2d_bytes_per_step": S * Tp * cfg.in_dim * 4,
                    "d2h_bytes_per_step": S * T * cfg.out_per_frame * 4, "ms_per_step": 1e3 * e2e_s / K},
            "gpu_launches": c_launches,
            "graph_launches": c_graphs,
            "repeats": repeats,
            "clocks": clocks,
            "roofline": roof,
            "kernels": kernels,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line))
    for s_ in streams:
        s_.close()
    model.destroy()
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Decode-throughput benchmark of the rollout-decoding library on synthetic self-play-shaped work.

One "step" is one call of spiral_decode_step over every concurrent game: embedding, all decoder
layers (RMSNorm, QKV, q/k-norm + RoPE + cache append, paged GQA attention, output projection,
SwiGLU MLP), LM head and the Gumbel-argmax draw, free-running (each sampled token is the next
input).  The default workload is the Qwen3-4B-shaped decoder with 128 concurrent games, each
with a 512-token context, decoding 256 tokens at temperature 1.0 with seeded Gumbel noise.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

prints one JSON line.  With N > 1 (launched by torch.distributed.run) every rank runs its own
set of games on its own GPU with replicated weights -- games are independent, nothing is
exchanged inside a step -- and the time is the maximum over ranks.
`--impl reference` times the CPU oracle (test infrastructure, never tuned) on a bounded sample of
the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

import synth  # noqa: E402

METRIC = "decode tokens/s at 1 B200 (Qwen3-4B shape, 128 games) and % of HBM roofline"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0            # the "~8 TB/s" the 70 % target is stated against
FALLBACK_HBM_GBS = 6650.0
FALLBACK_TENSOR_TFLOPS = 1400.0     # sustained dense 16-bit rate measured earlier on this kind of GPU
APPEND_TOKENS = 300                 # observation appended to every game between two turns (context-append measurement)
GUMBEL_RING = 8
# DRAM bytes (read + written) per algorithmic byte, from ncu captures of a 2-layer case of the same kernels
# (the attention kernel's traffic is whole 16-token pages of every game and grows in proportion to the
# cached tokens; a GEMM's is its weights once plus what leaves L2 of activations and partial sums).  None
# when a kernel has changed since its counters were taken.
ATTN_DRAM_PER_ALGORITHMIC_BYTE = 1.050
GEMM_DRAM_PER_ALGORITHMIC_BYTE = 1.050
MIN_TIMED_MS = 2000.0               # the timed window is repeated until this much GPU time has been timed
MAX_WINDOWS = 64
READ_CEILING_BYTES = 4 << 30        # buffer of the read-only bandwidth probe

WORKLOADS = {
    # name: (shape, games, context at the first timed step, default steps)
    "qwen3_4b_128games": ("qwen3_4b", 128, 512, 256),
    "llama31_8b_64seqs": ("llama31_8b", 64, 2560, 128),
    "qwen25_7b_64seqs_long": ("qwen25_7b", 64, 8192, 64),
    "tiny_4seqs": ("tiny", 4, 96, 32),
}


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="qwen3_4b_128games", choices=sorted(WORKLOADS))
    ap.add_argument("--games", type=int, default=None, help="override the number of concurrent games")
    ap.add_argument("--context", type=int, default=None, help="override the context at the first timed step")
    ap.add_argument("--layers", type=int, default=None, help="override the depth (profiling of small cases)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-kernel-times", action="store_true")
    ap.add_argument("--no-append", action="store_true", help="skip the context-append (prefill) measurement")
    ap.add_argument("--episode-config", action="store_true",
                    help="instead of the decode benchmark: the multi-turn episode configuration (256 games x 8 turns, "
                         "150-token observations, moves of 64-512 tokens) through the scheduler, one line of its own")
    ap.add_argument("--pool-gb", type=float, default=120.0, help="KV pool of --episode-config")
    ap.add_argument("--kv", default="f16", choices=["f16", "bf16"])
    ap.add_argument("--read-ceiling", action="store_true",
                    help="only measure the read-only bandwidth ceiling of the device (persistent TMA ring, no compute)")
    ap.add_argument("--no-read-ceiling", action="store_true")
    ap.add_argument("--min-timed-ms", type=float, default=MIN_TIMED_MS,
                    help="repeat the timed window until this much GPU time is timed (0: one window, for profiler runs)")
    return ap.parse_args()


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), "measured"
    return FALLBACK_HBM_GBS, "fallback"


def measured_tensor_peak():
    """Dense 16-bit tensor throughput a kernel inside a long pass can be held against (TFLOP/s)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            j = json.load(f)
        if "bf16_tflops_sustained" in j:
            return float(j["bf16_tflops_sustained"]), "measured (sustained)"
    return FALLBACK_TENSOR_TFLOPS, "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            self.f = os.fdopen(fd, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.gpu)], stdout=self.f,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.f.close()
        sm, smax, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                p = [x.strip() for x in line.split(",")]
                if len(p) < 9:
                    continue
                try:
                    sm.append(float(p[1])); smax.append(float(p[2])); power.append(float(p[3]))
                except ValueError:
                    continue
                for name, val in zip(names, p[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons),
                       samples=len(sm), power_w_max=max(power))
        return out


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        backend = "nccl" if torch.cuda.is_available() else "gloo"
        dist.init_process_group(backend=backend)
    return world, rank, local


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def max_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, world: int, device) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def workload_of(args):
    shape_name, games, context, steps = WORKLOADS[args.workload]
    desc = synth.shape(shape_name)
    if args.layers:
        desc["n_layers"] = args.layers
    games = args.games or games
    context = args.context or context
    steps = args.steps if args.steps is not None else steps
    return shape_name, desc, games, context, steps


def read_ceiling_gbs(sp, device_index, stream=None) -> float:
    """GB/s of a pure read stream: a persistent grid of one CTA per SM pulling 16 KB tiled TMA boxes through a
    6-stage shared-memory ring (the configuration that read fastest in a sweep of box sizes and depths), over a
    4 GB buffer, repeated to about a second; the best pass counts."""
    buf = torch.empty(READ_CEILING_BYTES, dtype=torch.uint8, device=torch.device("cuda", device_index))
    buf.zero_()
    torch.cuda.synchronize()
    sp.spiral_read_ceiling(device_index, buf, 16384, 6, 1, 0, True, 1, stream)
    best, spent = 0.0, 0.0
    while spent < 1.0:
        t0 = time.perf_counter()
        best = max(best, sp.spiral_read_ceiling(device_index, buf, 16384, 6, 1, 0, True, 4, stream))
        spent += time.perf_counter() - t0
    del buf
    return round(best, 1)


def kv_step_bytes(desc, lens_after_append) -> int:
    """K and V bytes the attention of one step has to read: every cached position of every game,
    the appended one included, over all layers."""
    return int(sum(lens_after_append)) * synth.kv_bytes_per_token(desc)


# ------------------------------------------------------------------------------------------------
# the library's arm
# ------------------------------------------------------------------------------------------------

def run_ours(args):
    world, rank, local = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device; the decode path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    import paper_2506_24119_b200 as sp

    shape_name, desc, n_games, context, steps = workload_of(args)
    warmup = args.warmup
    V = desc["vocab"]
    seed = synth.MASTER_SEED + 7919 * rank            # every rank plays its own games
    total_steps = warmup + steps
    start_len = context - warmup                      # the first TIMED step sees `context` cached tokens
    if start_len < 1:
        raise SystemExit("context must exceed warmup")
    max_ctx = context + max(steps, 0 if args.no_append else APPEND_TOKENS) + 16
    if not args.no_append:
        max_ctx = max(max_ctx, 2 * (APPEND_TOKENS + 64) + 16)      # the two-turn episodes of the scheduler pass

    w = synth.make_weights(desc, seed=synth.MASTER_SEED, device=dev)
    packed = sp.pack_weights(w)
    del w
    ctx = sp.spiral_init(desc, packed, local, max_batch=n_games, max_ctx=max_ctx)
    page_bytes = sp.spiral_kv_page_bytes(desc, 16)
    pages_per_game = (max_ctx + 15) // 16
    pool = torch.empty(n_games * pages_per_game * page_bytes, dtype=torch.uint8, device=dev)
    kv_dtype = sp.SPIRAL_KV_F16 if args.kv == "f16" else sp.SPIRAL_KV_BF16
    kv = sp.spiral_kv_alloc(ctx, pool, 16, n_games, max_ctx, kv_dtype)
    games = list(range(n_games))
    ids = (ctypes.c_int32 * n_games)(*games)

    # caches of `start_len` tokens per game: seeded random keys/values (same bytes per step as
    # prefilled ones; decouples the decode measurement from the prompt pass)
    Hkv, hd = desc["n_kv_heads"], desc["head_dim"]
    for layer in range(desc["n_layers"]):
        n = n_games * start_len * Hkv * hd
        k = synth.uniform_bf16(seed, 2 * layer, n, 2.0, dev).to(kv.dtype).view(n_games, start_len, Hkv, hd)
        v = synth.uniform_bf16(seed, 2 * layer + 1, n, 1.0, dev).to(kv.dtype).view(n_games, start_len, Hkv, hd)
        for g in games:
            sp.spiral_kv_load(ctx, kv, g, layer, k[g], v[g])
    torch.cuda.synchronize()
    del k, v

    ring = [synth.gumbel_noise(seed, s, n_games, V, dev) for s in range(GUMBEL_RING)]
    tok0 = synth.token_ids(seed, 1, n_games, V, dev)
    tok = [tok0.clone(), torch.empty_like(tok0)]
    # a stream of our own: the legacy default stream cannot be captured, and on any other stream
    # the library replays its recorded CUDA graph of the step
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(stream)

    def rewind():
        sp.spiral_kv_truncate(kv, games, [start_len] * n_games)
        tok[0].copy_(tok0)

    def decode_steps(first, count):
        for s in range(first, first + count):
            sp.spiral_decode_step(ctx, kv, ids, tok[s & 1], ring[s % GUMBEL_RING], 1.0, tok[(s + 1) & 1], None, stream)

    # ---- device-resident timing -------------------------------------------------------------
    # A window = warm-up steps (untimed) + exactly `steps` timed steps, bracketed by barrier + synchronize and
    # by CUDA events on the launch stream.  The window is repeated (games rolled back in between) until
    # MIN_TIMED_MS of GPU time have been timed; the line reports the median window and the spread.
    sp.spiral_profile(ctx, 0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler = ClockSampler(local)
    sampler.start()
    window_ms, launches, timed_ms = [], 0, 0.0
    while len(window_ms) < MAX_WINDOWS and (not window_ms or timed_ms < args.min_timed_ms):
        if window_ms:
            rewind()
        decode_steps(0, warmup)
        torch.cuda.synchronize(); barrier(world)
        launches0 = sp.spiral_launch_count(ctx)
        e0.record(stream)
        decode_steps(warmup, steps)
        e1.record(stream)
        torch.cuda.synchronize(); barrier(world)
        launches = sp.spiral_launch_count(ctx) - launches0
        window_ms.append(max_over_ranks(e0.elapsed_time(e1), world, dev))
        timed_ms += window_ms[-1]
    clocks = sampler.stop()
    rc, detail = sp.spiral_last_status(ctx)
    if rc != 0:
        raise SystemExit(f"device status {rc} ({detail}) after the timed region")
    srt = sorted(window_ms)
    ms_total = srt[len(srt) // 2] if len(srt) % 2 else 0.5 * (srt[len(srt) // 2 - 1] + srt[len(srt) // 2])
    ms_local = ms_total
    pct = lambda q: srt[min(len(srt) - 1, max(0, int(round(q * (len(srt) - 1)))))]
    windows = {"n": len(srt), "timed_ms_total": round(timed_ms, 1), "ms_per_step_median": round(ms_total / steps, 4),
               "ms_per_step_p10": round(pct(0.1) / steps, 4), "ms_per_step_p90": round(pct(0.9) / steps, 4),
               "ms_per_step_min": round(srt[0] / steps, 4), "ms_per_step_max": round(srt[-1] / steps, 4)}
    tokens_local = n_games * steps
    tokens_all = sum_over_ranks(tokens_local, world, dev)
    value = tokens_all / (ms_total * 1e-3)

    # bytes one rank's timed region has to read: weights every step + the growing caches
    wbytes = synth.weight_bytes_per_step(desc)
    kv_bytes = sum(kv_step_bytes(desc, [context + s + 1] * n_games) for s in range(steps))
    step_bytes_mean = wbytes + kv_bytes / steps
    achieved_step_gbs = (wbytes * steps + kv_bytes) / (ms_local * 1e-3) / 1e9
    peak, peak_kind = measured_peaks()

    # ---- what a pure read stream reaches on this device (the step reads weights and caches, writes next to nothing)
    read_ceiling = None
    if not args.no_read_ceiling:
        read_ceiling = read_ceiling_gbs(sp, local, stream)

    # ---- per-kernel times: same steps again with events around every launch ------------------
    roofline, kernels = None, None
    if not args.no_kernel_times:
        rewind()
        decode_steps(0, warmup)
        sp.spiral_profile(ctx, (1 << len(sp.KERNEL_CLASSES)) - 1)
        decode_steps(warmup, steps)
        kernels = {}
        tot = 0.0
        for c, name in enumerate(sp.KERNEL_CLASSES):
            ms, n = sp.spiral_profile_read(ctx, c)
            if n:
                kernels[name] = {"launches": n, "ms_total": round(ms, 3), "us_per_launch": round(1e3 * ms / n, 2)}
                tot += ms
        sp.spiral_profile(ctx, 0)
        L = desc["n_layers"]
        per_class_bytes = {
            "attn": kv_bytes,
            "qkv": 2 * L * steps * desc["d_model"] * (desc["n_q_heads"] + 2 * Hkv) * hd,
            "o": 2 * L * steps * desc["d_model"] * desc["n_q_heads"] * hd,
            "gate_up": 2 * L * steps * 2 * desc["d_model"] * desc["d_ff"],
            "down": 2 * L * steps * desc["d_model"] * desc["d_ff"],
            "lm_head": steps * (2 * V * desc["d_model"] + 4 * n_games * V),
        }
        for name, b in per_class_bytes.items():
            if name in kernels:
                k = kernels[name]
                k["gbs"] = round(b / (k["ms_total"] * 1e-3) / 1e9, 1)
                k["share_of_kernel_time"] = round(k["ms_total"] / tot, 4)
        # the dominant kernel once more with events around its launches only: with every kernel
        # bracketed the event records between kernels stretch each bracket by several microseconds
        rewind()
        decode_steps(0, warmup)
        sp.spiral_profile(ctx, 1 << sp.KERNEL_CLASSES.index("attn"))
        decode_steps(warmup, steps)
        ms, nl = sp.spiral_profile_read(ctx, sp.KERNEL_CLASSES.index("attn"))
        sp.spiral_profile(ctx, 0)
        a = {"ms_total": ms, "launches": nl, "us_per_launch": round(1e3 * ms / nl, 2)}
        achieved = kv_bytes / (a["ms_total"] * 1e-3) / 1e9
        roofline_attn = {"kernel": "attn_decode_kernel", "bound": "hbm", "achieved": round(achieved, 1),
                         "peak": peak, "unit": "GB/s", "frac": round(achieved / peak, 4), "peak_kind": f"of {peak_kind}",
                         "frac_of_read_ceiling": round(achieved / read_ceiling, 4) if read_ceiling else None,
                         "traffic": (int(ATTN_DRAM_PER_ALGORITHMIC_BYTE * kv_bytes / (steps * L))
                                     if ATTN_DRAM_PER_ALGORITHMIC_BYTE and shape_name == "qwen3_4b" else None),
                         "algorithmic_bytes_per_launch": int(kv_bytes / (steps * L)),
                         "us_per_launch": a["us_per_launch"], "launches": a["launches"]}
        # the four layer projections (one kernel function, four launches per layer: by function the largest share
        # of the step), bracketed alone in the same way; algorithmic bytes = their weight matrices, read once
        rewind()
        decode_steps(0, warmup)
        gemm_classes = ("qkv", "o", "gate_up", "down")
        sp.spiral_profile(ctx, sum(1 << sp.KERNEL_CLASSES.index(c) for c in gemm_classes))
        decode_steps(warmup, steps)
        g_ms, g_n = 0.0, 0
        for c in gemm_classes:
            ms_c, n_c = sp.spiral_profile_read(ctx, sp.KERNEL_CLASSES.index(c))
            g_ms += ms_c
            g_n += n_c
        sp.spiral_profile(ctx, 0)
        g_bytes = sum(per_class_bytes[c] for c in gemm_classes)
        g_ach = g_bytes / (g_ms * 1e-3) / 1e9
        roofline = {"kernel": "tc_gemm_kernel<0> (QKV, output, gate/up and down projections)", "bound": "hbm",
                    "achieved": round(g_ach, 1), "peak": peak, "unit": "GB/s", "frac": round(g_ach / peak, 4),
                    "peak_kind": f"of {peak_kind}",
                    "frac_of_read_ceiling": round(g_ach / read_ceiling, 4) if read_ceiling else None,
                    "read_ceiling_gbs": read_ceiling,
                    "traffic": (int(GEMM_DRAM_PER_ALGORITHMIC_BYTE * g_bytes / g_n)
                                if GEMM_DRAM_PER_ALGORITHMIC_BYTE and shape_name == "qwen3_4b" else None),
                    "algorithmic_bytes_per_launch": int(g_bytes / g_n), "us_per_launch": round(1e3 * g_ms / g_n, 2),
                    "launches": g_n, "share_of_kernel_time": round(sum(kernels[c]["ms_total"] for c in gemm_classes) / tot, 4),
                    "attention": roofline_attn}

    # ---- end to end: host buffers in, host tokens out, through the public call ---------------
    e2e = None
    if not args.no_e2e:
        rewind()
        h_ring = [r.cpu().pin_memory() for r in ring]
        h_tok = [tok0.cpu().pin_memory(), torch.empty(n_games, dtype=torch.int32).pin_memory()]

        def host_steps(first, count):
            for s in range(first, first + count):
                sp.spiral_decode_step_host(ctx, kv, ids, h_tok[s & 1], h_ring[s % GUMBEL_RING], 1.0,
                                           h_tok[(s + 1) & 1], stream)
        host_steps(0, warmup)
        torch.cuda.synchronize(); barrier(world)
        e0.record(stream)
        host_steps(warmup, steps)
        e1.record(stream)
        torch.cuda.synchronize(); barrier(world)
        ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev)
        e2e = {"value": round(tokens_all / (ms_e2e * 1e-3), 1), "unit": UNIT,
               "h2d_bytes_per_step": n_games * 4 + n_games * V * 4, "d2h_bytes_per_step": n_games * 4,
               "ms_per_step": round(ms_e2e / steps, 4)}
        del h_ring

    # ---- context append: the observation every game receives between two turns ---------------
    # (reported beside the decode metric, outside its timed region: APPEND_TOKENS new tokens per game
    # on top of the decode workload's caches, through the public call, device-resident tokens)
    append = None
    if not args.no_append:
        new_tok = synth.token_ids(seed, 77, n_games * APPEND_TOKENS, V, dev)
        offs = [i * APPEND_TOKENS for i in range(n_games + 1)]
        times = []
        for r in range(3):                      # the first call allocates the path's workspace
            rewind()
            torch.cuda.synchronize(); barrier(world)
            e0.record(stream)
            sp.spiral_prefill(ctx, kv, games, new_tok, offs, None, stream)
            e1.record(stream)
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms_app = max_over_ranks(min(times[1:]), world, dev)
        rewind()
        sp.spiral_profile(ctx, (1 << len(sp.KERNEL_CLASSES)) - 1)
        sp.spiral_prefill(ctx, kv, games, new_tok, offs, None, stream)
        torch.cuda.synchronize()
        cls = {name: sp.spiral_profile_read(ctx, c)[0] for c, name in enumerate(sp.KERNEL_CLASSES)}
        sp.spiral_profile(ctx, 0)
        L, D, F, Hq = desc["n_layers"], desc["d_model"], desc["d_ff"], desc["n_q_heads"]
        n_new = n_games * APPEND_TOKENS
        gemm_flop = 2.0 * n_new * L * (D * (Hq + 2 * Hkv) * hd + Hq * hd * D + 3 * D * F)
        keys = sum(start_len + i + 1 for i in range(APPEND_TOKENS))         # keys seen by one game's new queries
        attn_flop = 4.0 * n_games * L * Hq * hd * keys
        tensor_peak = measured_tensor_peak()
        gemm_ms = sum(cls[k] for k in ("qkv", "o", "gate_up", "down"))
        append = {"new_tokens_per_game": APPEND_TOKENS, "context_before": start_len, "ms": round(ms_app, 2),
                  "tokens_per_s": round(sum_over_ranks(n_new, world, dev) / (ms_app * 1e-3), 1),
                  "tflops_whole_pass": round((gemm_flop + attn_flop) / (ms_app * 1e-3) / 1e12, 1),
                  "gemm": {"bound": "tensor", "achieved": round(gemm_flop / (gemm_ms * 1e-3) / 1e12, 1),
                           "peak": tensor_peak[0], "unit": "TFLOP/s", "peak_kind": f"of {tensor_peak[1]}",
                           "frac": round(gemm_flop / (gemm_ms * 1e-3) / 1e12 / tensor_peak[0], 4),
                           "ms_event_bracketed": round(gemm_ms, 2)},
                  "attention": {"tflops": round(attn_flop / (cls["attn"] * 1e-3) / 1e12, 1),
                                "ms_event_bracketed": round(cls["attn"], 2),
                                "pipe": "mma.sync" if os.environ.get("SPIRAL_APPEND_ATTN", "")[:1] == "m" else "tcgen05"}}

    # ---- evaluation-style decoding: the same step ending in the nucleus sampler (T 0.6, top-p 0.95) ----
    nucleus = None
    if not args.no_append:
        rewind()
        n_eval = min(steps, 32)

        def nucleus_steps(first, count):
            for s in range(first, first + count):
                sp.spiral_decode_step_nucleus(ctx, kv, ids, tok[s & 1], ring[s % GUMBEL_RING], 0.6, 0.95, tok[(s + 1) & 1],
                                              None, stream)
        nucleus_steps(0, warmup)
        torch.cuda.synchronize(); barrier(world)
        e0.record(stream)
        nucleus_steps(warmup, n_eval)
        e1.record(stream)
        torch.cuda.synchronize()
        ms_nuc = max_over_ranks(e0.elapsed_time(e1), world, dev)
        nucleus = {"temperature": 0.6, "top_p": 0.95, "steps": n_eval, "ms_per_step": round(ms_nuc / n_eval, 4),
                   "tokens_per_s": round(sum_over_ranks(n_games * n_eval, world, dev) / (ms_nuc * 1e-3), 1)}

    # ---- episodes through the scheduler: more games than batch rows, two turns each, ragged budgets ----
    episodes = None
    if not args.no_append:
        sp.spiral_kv_release(kv, games)
        sched = sp.spiral_sched_create(ctx, kv, -1)
        n_ep = n_games                      # one wave of games per cache row, each two turns
        obs_len = synth.lengths(seed, 91, 2 * n_ep, 150, APPEND_TOKENS)
        budget = synth.lengths(seed, 92, 2 * n_ep, 16, 64)
        handles = [sp.spiral_sched_open(sched) for _ in range(n_ep)]
        turn = {g: 0 for g in handles}
        for i, g in enumerate(handles):
            sp.spiral_sched_turn(sched, g, synth.token_ids(seed, 500 + i, obs_len[i], V).tolist(), budget[i])
        open_turns, ticks = n_ep, 0
        torch.cuda.synchronize(); barrier(world)
        t0 = time.perf_counter()
        e0.record(stream)
        while open_turns:
            sp.spiral_sched_tick(sched, ring[ticks % GUMBEL_RING], 1.0, stream)
            ticks += 1
            while True:
                done = sp.spiral_sched_poll(sched)
                if done is None:
                    break
                g = done[0]
                turn[g] += 1
                open_turns -= 1
                if turn[g] < 2:
                    i = n_ep + handles.index(g)
                    sp.spiral_sched_turn(sched, g, synth.token_ids(seed, 500 + i, obs_len[i], V).tolist(), budget[i])
                    open_turns += 1
        e1.record(stream)
        torch.cuda.synchronize()
        ms_ep = max_over_ranks(e0.elapsed_time(e1), world, dev)
        st = sp.spiral_sched_stats(sched)
        episodes = {"games": n_ep, "turns_per_game": 2, "ticks": ticks, "ms": round(ms_ep, 1),
                    "wall_ms": round((time.perf_counter() - t0) * 1e3, 1),
                    "appended_tokens": st["appended"], "decoded_tokens": st["decoded"], "dropped_samples": st["dropped"],
                    "decoded_tokens_per_s": round(sum_over_ranks(st["decoded"], world, dev) / (ms_ep * 1e-3), 1),
                    "all_tokens_per_s": round(sum_over_ranks(st["decoded"] + st["appended"], world, dev) / (ms_ep * 1e-3), 1)}
        for g in handles:
            sp.spiral_sched_close(sched, g)
        sp.spiral_sched_free(sched)

    sp.spiral_free(ctx, kv)

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu_baseline = oracle_sample_rate(desc, context, budget_s=20.0, dev=dev)

    if rank == 0:
        line = {
            "metric": METRIC, "value": round(value, 1), "unit": UNIT, "n_gpus": world, "steps": steps,
            "warmup": warmup, "ms_per_step": round(ms_total / steps, 4), "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16 x bf16 -> f32", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape_name, "games_per_gpu": n_games,
                       "context_first_timed_step": context, "decode_steps": steps, "page_size": 16,
                       "kv_dtype": args.kv, "temperature": 1.0, "layers": desc["n_layers"],
                       "l2": "inputs larger than L2 (weights + caches of one step exceed 126 MB many times over)",
                       "timing": f"median of {windows['n']} windows of {steps} steps (repeated to >= {args.min_timed_ms / 1e3:.0f} s of GPU time)",
                       "parallelism": "replicas" if world > 1 else "single GPU"},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "windows": windows,
            "step_roofline": {"bytes_per_step_mean": int(step_bytes_mean), "weight_bytes": wbytes,
                              "achieved_gbs": round(achieved_step_gbs, 1),
                              "frac_of_8TBs": round(achieved_step_gbs / NOMINAL_HBM_GBS, 4),
                              f"frac_of_{peak_kind}": round(achieved_step_gbs / peak, 4),
                              "read_ceiling_gbs": read_ceiling,
                              "frac_of_read_ceiling": round(achieved_step_gbs / read_ceiling, 4) if read_ceiling else None},
            "roofline": roofline, "kernels": kernels, "e2e": e2e, "cpu_baseline": cpu_baseline, "append": append,
            "nucleus_decoding": nucleus, "episodes": episodes,
        }
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------------------
# the CPU oracle, timed as it stands
# ------------------------------------------------------------------------------------------------

def oracle_setup(desc, context, n_games, dev, keep_layers=None):
    """Oracle model (optionally only its first keep_layers layers) + caches of `context` seeded
    random cached tokens for n_games games."""
    from oracle import oracle
    oracle.build()
    gen_dev = dev if dev is not None else "cpu"
    d = dict(desc)
    if keep_layers:
        d["n_layers"] = keep_layers
    w = synth.make_weights(d, seed=synth.MASTER_SEED, device=gen_dev)
    w = {k: ([t.cpu() if t is not None else None for t in v] if isinstance(v, list)
             else (v.cpu() if v is not None else None)) for k, v in w.items()}
    model = oracle.Model(d, w)
    Hkv, hd = d["n_kv_heads"], d["head_dim"]
    caches = []
    for g in range(n_games):
        c = model.new_cache(context + 1024)
        for layer in range(d["n_layers"]):
            k, v = synth.synthetic_kv(synth.MASTER_SEED, g, layer, context, Hkv, hd, gen_dev)
            c.load(layer, k.cpu(), v.cpu())
        c.set_len(context)
        caches.append(c)
    return oracle, model, caches, w


def oracle_token(oracle, model, cache, tok, step, V):
    """One game-token of the oracle: decode step + Gumbel-max draw.  Returns seconds."""
    noise = synth.gumbel_noise(synth.MASTER_SEED, step, 1, V)[0].numpy()
    t0 = time.perf_counter()
    lg = model.decode_step(cache, tok)
    oracle.sample(lg, noise, 1.0)
    return time.perf_counter() - t0


def oracle_sample_rate(desc, context, budget_s, dev):
    """Tokens/s of the oracle on a bounded sample: a few games of the same shape and context,
    decoded token by token until about budget_s seconds of CPU work are spent."""
    n_games = 2
    oracle, model, caches, _ = oracle_setup(desc, context, n_games, dev)
    V = desc["vocab"]
    toks = synth.token_ids(synth.MASTER_SEED, 3, 4096, V).tolist()
    oracle_token(oracle, model, caches[0], toks[0], 0, V)        # touch the weights once, untimed
    done, el = 0, 0.0
    while el < budget_s and done < 64:
        for g in range(n_games):
            el += oracle_token(oracle, model, caches[g], toks[(done + g) % 4096], done + g, V)
        done += n_games
    return {"value": round(done / el, 4), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
            "sample": f"{done} game-tokens: {n_games} games of the same shape at context {context}, "
                      f"decoded and sampled one token at a time in {el:.1f} s"}


def run_reference(args):
    """The oracle as the reference arm.  A step here is ONE game-token (the oracle decodes one game
    at a time); when warmup + steps tokens of the full-depth model would not end within a few
    minutes, each step runs the first `keep` layers only and the layer part of its time is scaled
    by layers / keep (layers are identical in shape, so their cost is linear in depth)."""
    world, rank, local = dist_setup(args.gpus)
    if rank != 0:
        return
    shape_name, desc, n_games, context, steps = workload_of(args)
    dev = torch.device("cuda", local) if torch.cuda.is_available() else None
    V, L = desc["vocab"], desc["n_layers"]
    toks = synth.token_ids(synth.MASTER_SEED, 3, 4096, V).tolist()
    warmup = args.warmup
    budget = 200.0
    # size the sample on a 2-layer probe: seconds per layer and for the head + sampler
    oracle, probe, pc, _ = oracle_setup(desc, context, 1, dev, keep_layers=min(2, L))
    oracle_token(oracle, probe, pc[0], toks[0], 0, V)
    t_probe = oracle_token(oracle, probe, pc[0], toks[1], 1, V)
    import numpy as np
    noise = synth.gumbel_noise(synth.MASTER_SEED, 0, 1, V)[0].numpy()
    t0 = time.perf_counter()
    hidden = probe.decode_step(pc[0], toks[2], want_logits=False, want_hidden=True)[1]
    t_layers_probe = time.perf_counter() - t0
    t_head = max(0.0, t_probe - t_layers_probe)
    t_layer = t_layers_probe / min(2, L)
    keep = L
    if (warmup + steps) * (t_layer * L + t_head) > budget:
        keep = int((budget / (warmup + steps) - t_head) / t_layer)
        keep = max(1, min(L, keep))
    del probe, pc
    oracle, model, caches, _ = oracle_setup(desc, context, 1, dev, keep_layers=keep)
    scale = L / keep

    def step_seconds(s):
        t = oracle_token(oracle, model, caches[0], toks[s % 4096], s, V)
        return (t - t_head) * scale + t_head if keep != L else t

    for s in range(warmup):
        step_seconds(s)
    total = sum(step_seconds(s) for s in range(warmup, warmup + steps))
    value = steps / total
    note = "" if keep == L else (f"; each step runs layers 0..{keep - 1} of {L} and the layer part of its time "
                                 f"(all but {t_head * 1e3:.0f} ms of LM head + sampler) is scaled by {scale:.2f}")
    sample = (f"each step = 1 game-token of the {shape_name} shape at context {context}+, decoded and sampled "
              f"by the oracle{note}")
    line = {"impl": "reference", "metric": METRIC, "value": round(value, 4), "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": round(1e3 * total / steps, 2),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": args.workload, "shape": shape_name, "games_per_gpu": n_games,
                       "context_first_timed_step": context, "decode_steps": steps, "layers": L},
            "cpu_baseline": {"value": round(value, 4), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                             "sample": sample},
            "e2e": {"value": round(value, 4), "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def run_episode_config(args):
    """Multi-turn self-play episodes on the Qwen3-4B shape through the scheduler: 256 games of 8 turns, a
    150-token observation and a move of uniform length in [64, 512] per turn, finished games leave.  The pool
    is what --pool-gb allows, below the games' worst case, so later turns wait for pages."""
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    import paper_2506_24119_b200 as sp
    desc = synth.shape("qwen3_4b")
    if args.layers:
        desc = dict(desc, n_layers=args.layers)
    n_games = args.games or 256
    n_turns, obs_len, lo, hi = 8, 150, 64, 512
    V = desc["vocab"]
    max_ctx = n_turns * (obs_len + hi) + 16
    w = synth.make_weights(desc, seed=synth.MASTER_SEED, device=dev)
    packed = sp.pack_weights(w)
    del w
    ctx = sp.spiral_init(desc, packed, 0, max_batch=n_games, max_ctx=max_ctx)
    page_bytes = sp.spiral_kv_page_bytes(desc, 16)
    n_pages = min(int(args.pool_gb * 1e9) // page_bytes, n_games * ((max_ctx + 15) // 16))
    pool = torch.empty(n_pages * page_bytes, dtype=torch.uint8, device=dev)
    kv = sp.spiral_kv_alloc(ctx, pool, 16, n_games, max_ctx, sp.SPIRAL_KV_F16)
    sched = sp.spiral_sched_create(ctx, kv, -1)
    seed = synth.MASTER_SEED
    budget = [synth.lengths(seed, 30 + t, n_games, lo, hi) for t in range(n_turns)]
    ring = [synth.gumbel_noise(seed, s, n_games, V, dev) for s in range(GUMBEL_RING)]
    stream = torch.cuda.Stream()
    torch.cuda.synchronize()
    torch.cuda.set_stream(stream)
    games = [sp.spiral_sched_open(sched) for _ in range(n_games)]
    turn_of = {g: 0 for g in games}

    def queue_turn(g):
        t = turn_of[g]
        sp.spiral_sched_turn(sched, g, synth.token_ids(seed, 1000 * t + g, obs_len, V).tolist(), budget[t][g])
    for g in games:
        queue_turn(g)
    left, ticks, most_waiting, running_sum = n_games, 0, 0, 0
    # roofline of the run, summed as it goes: per tick the weights are read once (or the batch's flops are done,
    # whichever takes longer), every decoded token reads its game's cache, every appended token costs its flops
    peak_bw = measured_peaks()[0] * 1e9
    peak_fl = measured_tensor_peak()[0] * 1e12
    wbytes = synth.weight_bytes_per_step(desc)
    params_flop = 2.0 * (wbytes / 2)                    # 2 flops per weight element and batch row
    kvb = synth.kv_bytes_per_token(desc)
    t_roof_weights, kv_read_bytes, append_flop = 0.0, 0.0, 0.0
    sampler = ClockSampler(0)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    sampler.start()
    t0 = time.perf_counter()
    e0.record(stream)
    while left:
        n = sp.spiral_sched_tick(sched, ring[ticks % GUMBEL_RING], 1.0, stream)
        ticks += 1
        running_sum += n
        if n > 0:
            t_roof_weights += max(wbytes / peak_bw, params_flop * n / peak_fl)
        if ticks % 64 == 0:
            most_waiting = max(most_waiting, sp.spiral_sched_stats(sched)["waiting"])
        while True:
            done = sp.spiral_sched_poll(sched)
            if done is None:
                break
            g = done[0]
            r = len(done[1])
            ctx_end = sp.spiral_kv_seq_len(kv, g)       # observation and response cached (the last token possibly not yet)
            kv_read_bytes += kvb * (r * ctx_end - r * (r - 1) / 2.0)
            append_flop += params_flop * obs_len + 4.0 * desc["n_layers"] * desc["n_q_heads"] * desc["head_dim"] * obs_len * (ctx_end - r)
            turn_of[g] += 1
            if turn_of[g] < n_turns:
                queue_turn(g)
            else:
                sp.spiral_sched_close(sched, g)
                left -= 1
    e1.record(stream)
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1)
    wall = (time.perf_counter() - t0) * 1e3
    clocks = sampler.stop()
    st = sp.spiral_sched_stats(sched)
    rc, detail = sp.spiral_last_status(ctx)
    if rc != 0:
        raise SystemExit(f"device status {rc} ({detail})")
    sp.spiral_sched_free(sched)
    sp.spiral_free(ctx, kv)
    t_roof = t_roof_weights + kv_read_bytes / peak_bw + append_flop / peak_fl
    print(json.dumps({
        "metric": "multi-turn episode tokens/s at 1 B200 (Qwen3-4B shape, 256 games x 8 turns)", "unit": "tokens/s",
        "roofline": {"t_roof_ms": round(t_roof * 1e3, 1), "frac": round(t_roof * 1e3 / ms, 4),
                     "formula": "sum over ticks max(W / BW, 2 B params / peak) + KV bytes read / BW + append flops / peak",
                     "decode_weights_or_flops_ms": round(t_roof_weights * 1e3, 1),
                     "kv_read_ms": round(kv_read_bytes / peak_bw * 1e3, 1), "append_ms": round(append_flop / peak_fl * 1e3, 1),
                     "bw_gbs": measured_peaks()[0], "tensor_tflops": measured_tensor_peak()[0], "peaks": "of measured"},
        "value": round((st["decoded"] + st["appended"]) / (ms * 1e-3), 1),
        "decoded_tokens_per_s": round(st["decoded"] / (ms * 1e-3), 1), "n_gpus": 1, "higher_is_better": True,
        "ms": round(ms, 1), "wall_ms": round(wall, 1), "ticks": ticks, "mean_games_per_tick": round(running_sum / ticks, 1),
        "decoded_tokens": st["decoded"], "appended_tokens": st["appended"], "dropped_samples": st["dropped"],
        "most_turns_waiting": most_waiting, "data": "synthetic", "dtype": "f16 x bf16 -> f32",
        "config": {"workload": "qwen3_4b_256games_8turns", "games": n_games, "turns": n_turns, "observation_tokens": obs_len,
                   "move_tokens": [lo, hi], "page_size": 16, "pool_pages": int(n_pages),
                   "worst_case_pages": n_games * ((max_ctx + 15) // 16), "layers": desc["n_layers"]},
        "clocks": clocks}))


def run_read_ceiling(args):
    torch.cuda.set_device(0)
    import paper_2506_24119_b200 as sp
    sampler = ClockSampler(0)
    sampler.start()
    gbs = read_ceiling_gbs(sp, 0)
    clocks = sampler.stop()
    peak, kind = measured_peaks()
    print(json.dumps({"metric": "read-only HBM bandwidth (persistent TMA ring, no compute)", "value": gbs, "unit": "GB/s",
                      "n_gpus": 1, "higher_is_better": True, "copy_peak_gbs": peak, "copy_peak_kind": kind,
                      "config": {"workload": "read_ceiling", "buffer_bytes": READ_CEILING_BYTES, "box_bytes": 16384,
                                 "stages": 6, "ctas_per_sm": 1, "tiled": True}, "clocks": clocks}))


def main():
    args = parse()
    if args.read_ceiling:
        return run_read_ceiling(args)
    if args.episode_config:
        return run_episode_config(args)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

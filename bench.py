#!/usr/bin/env python
"""Benchmark of the TiDAR decode step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 8b|1.5b|tiny] [--impl ours|reference]

A "step" is one pass of the whole decode path (slot assembly, every layer, LM
head with argmax, draft/verify/select, KV commit) for one sequence.  Prints ONE
JSON line.  Metric: decode tokens/s under a seeded acceptance-length schedule
(mean 8 at k = 16); the step cost does not depend on the acceptance length, so
the per-length table is tokens/s = L / latency.

``--impl reference`` times the CPU oracle (the only reference this method has) on
a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from tidar_synth import CONFIGS, acceptance_schedule, gen_model_weights, gen_token_ids, tensor_id

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}
SCHEDULE_SEED = 1234


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------
# algorithmic cost of one step (per sequence)
# ----------------------------------------------------------------------------
def step_cost(sh, k, n, n_layers=None, batch=1):
    """Algorithmic bytes and flops of one decode step of `batch` sequences with n cached positions each.

    bytes: every projection weight and the LM head once (bf16) + the K/V of the n
    cached positions once per layer.  flops: 2*T*params for the projections +
    4*T*Hq*hd*(keys visible per row) for attention.
    """
    T = k * (k + 1)
    L = n_layers or sh.n_layers
    per_layer = (sh.d_model * (sh.n_q_heads + 2 * sh.n_kv_heads) * sh.head_dim + sh.n_q_heads * sh.head_dim * sh.d_model
                 + 3 * sh.d_model * sh.d_ffn)
    params = L * per_layer + sh.vocab * sh.d_model
    kv_bytes = n * L * 2 * sh.n_kv_heads * sh.head_dim * 2
    # keys per row: causal j sees n+j+1, mask (b, .) sees n+b+1+k
    keys = sum(n + j + 1 for j in range(k)) + sum(k * (n + b + 1 + k) for b in range(k))
    attn_flops = L * 4 * sh.n_q_heads * sh.head_dim * keys
    kv_bytes *= batch; attn_flops *= batch; T *= batch      # weights are shared, everything else is per sequence
    return {"T": T, "params": params, "weight_bytes": 2 * params, "kv_bytes": kv_bytes,
            "gemm_flops": 2 * T * params, "attn_flops": attn_flops,
            "bytes": 2 * params + kv_bytes, "flops": 2 * T * params + attn_flops}


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.idx, self.p = gpu_index, None

    def __enter__(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(self.idx), f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                       "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.p = None
        return self

    def __exit__(self, *a):
        self.out = ""
        if self.p is not None:
            self.p.terminate()
            try:
                self.out, _ = self.p.communicate(timeout=5)
            except Exception:
                self.p.kill()

    def summary(self):
        sm, mx, reasons, pw = [], [], set(), []
        for line in self.out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); pw.append(float(f[3]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        # samples under load = upper half of the clock samples' power
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons), "samples": len(sm),
                "power_w_max": max(pw)}


# ----------------------------------------------------------------------------
# CPU oracle: one whole decode step, timed
# ----------------------------------------------------------------------------
def pipelined_steps(t, seqs, forced_per_step):
    """Runs the steps through tidar_step_async / tidar_step_wait with two steps in flight (every length is
    forced, so the next step is enqueued while the previous one runs and the device never waits for the
    host); returns the tokens emitted."""
    tokens, in_flight = 0, 0
    for f in forced_per_step:
        t.step_async(seqs, f)
        in_flight += 1
        if in_flight == 2:
            _, L = t.step_wait(); tokens += sum(L); in_flight -= 1
    while in_flight:
        _, L = t.step_wait(); tokens += sum(L); in_flight -= 1
    return tokens


def oracle_step_timed(sh, k, n, n_steps=1):
    """Times `n_steps` full decode steps of the CPU oracle (every layer, the whole LM head, acceptance,
    selection, commit) for one sequence with n cached positions.

    The oracle runs as it stands (float64 NumPy on the host cores).  Its weights are the generator's,
    handed over one layer at a time (produced on the GPU when there is one, else on the host) so that
    the host never holds more than one layer in float64; the time spent producing them is measured
    and NOT counted.  The cache holds seeded random K/V (timing does not depend on the values).
    Returns (seconds per step, seconds spent producing weights per step).
    """
    from oracle import tidar_oracle as O
    from tidar_synth import lazy_model_weights, production_seconds
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = lazy_model_weights(sh, dev)
    cfg = O.OracleConfig(sh.n_layers, sh.d_model, sh.n_q_heads, sh.n_kv_heads, sh.head_dim, sh.d_ffn, sh.vocab, sh.rope_theta,
                         sh.rms_eps, sh.mask_token_id, 1.0)
    rng = np.random.default_rng(sh.seed)
    block = gen_token_ids(sh.seed, tensor_id("drafts"), k, sh.vocab - 1).numpy().astype(np.int64)
    st = O.OracleState(n=n, k_cache=[rng.standard_normal((n, sh.n_kv_heads, sh.head_dim)) for _ in range(sh.n_layers)],
                       v_cache=[rng.standard_normal((n, sh.n_kv_heads, sh.head_dim)) for _ in range(sh.n_layers)], block=block)
    total, gen = 0.0, 0.0
    for _ in range(n_steps):
        g0 = production_seconds()
        t0 = time.perf_counter()
        O.step(cfg, w, st)
        dt = time.perf_counter() - t0
        dg = production_seconds() - g0
        total += dt - dg; gen += dg
    return total / n_steps, gen / n_steps


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else os.cpu_count()
    except Exception:
        return os.cpu_count()


# ----------------------------------------------------------------------------
def run_reference(args, sh, k, n0):
    """The reference arm: the CPU oracle on this workload.  A full 8B-class oracle step takes ~10 s of
    float64 arithmetic, so the arm times a bounded number of whole steps (one by default) whatever
    --steps says, and reports that number as `steps`."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    n_timed = max(1, min(args.steps, args.ref_steps))
    step_s, gen_s = oracle_step_timed(sh, k, n0, n_timed)
    mean_L = float(acceptance_schedule(SCHEDULE_SEED, 4096, k).numpy().mean())
    value = mean_L / step_s
    cores = blas_threads()
    sample = (f"{n_timed} whole decode step(s) of the unmodified oracle (all {sh.n_layers} layers, full LM head, k={k}, {k*(k+1)} slots, "
              f"n={n0} cached positions, float64 NumPy); weights handed over layer by layer, their production "
              f"({gen_s:.1f} s per step) not counted; tokens/s = mean schedule acceptance {mean_L:.2f} / step time")
    cfgd = workload_config(sh, k, n0, 1)
    cfgd["reference_steps_timed"] = n_timed
    cfgd["reference_steps_requested"] = args.steps
    line = {"impl": "reference", "metric": "decode_tokens_per_s", "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
            "steps": n_timed, "warmup": 0, "ms_per_step": 1e3 * step_s,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": cfgd, "extrapolated": False,
            "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample, "extrapolated": False},
            "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line))


def attention_microbench(reps=50):
    """Structured-mask attention alone (`tidar_attention`: row table, attention kernel, merge of the key
    splits) at 32/8 heads, head_dim 128, k = 16 and 1 k .. 32 k cached positions in shuffled pages; one
    JSON line per length.  A diagnostic beside the step benchmark, not a bench value."""
    from dataclasses import replace
    from paper_2511_08923_b200 import Tidar, pack_weights
    hd, Hq, Hkv, k = 128, 32, 8, 16
    sh = replace(CONFIGS["tiny"], head_dim=hd, n_q_heads=Hq, n_kv_heads=Hkv, n_layers=1, vocab=64, d_ffn=64, d_model=64)
    t = Tidar(sh, pack_weights(gen_model_weights(sh), "cuda:0"), k_max=k, max_batch=1, max_seq_len=128, impl=0)
    T = k * (k + 1)
    pk, _ = peaks()
    g = torch.Generator(device="cuda:0"); g.manual_seed(7)
    rnd = lambda *shape: torch.randn(*shape, device="cuda:0", generator=g).bfloat16()
    for n in (1024, 4096, 16384, 32768):
        pps = (n + k + 63) // 64
        q, kp, vp, kl, vl = rnd(T, Hq, hd), rnd(pps, Hkv, 64, hd), rnd(pps, Hkv, 64, hd), rnd(k * k, Hkv, hd), rnd(k * k, Hkv, hd)
        pt = torch.randperm(pps, device="cuda:0", generator=g).to(torch.int32).view(1, pps)
        sl = torch.tensor([n], dtype=torch.int32, device="cuda:0")
        out = torch.empty(T, Hq * hd, dtype=torch.bfloat16, device="cuda:0")
        for _ in range(3):
            t.attention(q, kp, vp, pt, sl, kl, vl, out, 1, k)
        t.sync()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            t.attention(q, kp, vp, pt, sl, kl, vl, out, 1, k)
        e1.record(); torch.cuda.synchronize()
        us = e0.elapsed_time(e1) / reps * 1e3
        # skipped-tile evidence: key tiles the kernel's CTAs visit in one call, against a dense mask
        # (every 128-row query tile of every KV head against every 64-key tile of [cache | step slots])
        t.count_attention_tiles(True)
        t.attention(q, kp, vp, pt, sl, kl, vl, out, 1, k)
        visited = t.count_attention_tiles(False)
        spt = 128 // (Hq // Hkv)
        q_tiles = (T + spt - 1) // spt
        dense = Hkv * q_tiles * ((n + k + 63) // 64 + (k * k + 63) // 64)
        local_blocks = (2 * k + 1) / float((k + 1) ** 2)
        # the cached part is dense for every row; what the mask's block structure saves is in the step-local part
        cache_tiles = 0
        for qt in range(q_tiles):
            slots = range(qt * spt, min((qt + 1) * spt, T))
            nvis = max(n + s_ + 1 if s_ < k else n + (s_ - k) // k + 1 for s_ in slots)
            cache_tiles += (nvis + 63) // 64
        local_visited = visited - Hkv * cache_tiles
        local_dense = Hkv * q_tiles * ((k * k + 63) // 64)
        keys = sum(n + j + 1 for j in range(k)) + sum(k * (n + b + 1 + k) for b in range(k))
        flops, nbytes = 4 * Hq * hd * keys, n * Hkv * hd * 2 * 2
        print(json.dumps({"attention_microbench": {"cached_positions": n, "k": k, "heads": f"{Hq}/{Hkv}", "head_dim": hd},
                          "us_per_call": round(us, 1), "tflops": round(flops / us / 1e6, 1), "kv_gbs": round(nbytes / us / 1e3, 1),
                          "frac_of_measured_bf16_peak": round(flops / us / 1e6 / pk["bf16_tflops_sustained"], 3),
                          "key_tiles_visited": visited, "key_tiles_dense_mask": dense, "skipped_tile_frac": round(1.0 - visited / dense, 4),
                          "local_tiles_visited": local_visited, "local_tiles_dense_mask": local_dense,
                          "local_skipped_tile_frac": round(1.0 - local_visited / local_dense, 4),
                          "local_kxk_subblocks_nonempty_frac": round(local_blocks, 4)}))
    t.close()


def measure_classes(t, seqs, forced_L, impl, n_t=4):
    """Per-class kernel time of a step (ms): (timeline in graph mode, CUDA events around plain launches)."""
    cls, cls_plain = {}, {}
    if impl == 0:
        t.set_timeline(True)
        t.step(seqs, forced_L)                        # re-captures the graph with the stamps in
        for _ in range(n_t):
            t.step(seqs, forced_L)
            for kk, v in t.timeline().items():
                cls[kk] = cls.get(kk, 0.0) + v / n_t
        t.set_timeline(False)
    t.set_timing(True)
    for _ in range(n_t):
        t.step(seqs, forced_L)
        for kk, v in t.timing().items():
            cls_plain[kk] = cls_plain.get(kk, 0.0) + v / n_t
    t.set_timing(False)
    if not cls:
        cls = dict(cls_plain)
    return cls, cls_plain


def measure_other_workload(sh, impl, dev, stream, steps=64, warmup=5):
    """One more model class in the same run: build it, prefill, time `steps` decode steps under the
    schedule (CUDA events on the library's stream), per-class kernel time, roofline fractions."""
    from paper_2511_08923_b200 import Tidar, pack_weights
    k, n0 = sh.k, sh.prompt_len
    packed = pack_weights(gen_model_weights(sh, device=dev), dev)
    t = Tidar(sh, packed, k_max=k, max_batch=1, max_seq_len=n0 + (steps + warmup + 16) * k + 64, impl=impl, device=dev, stream=stream)
    prompt = gen_token_ids(sh.seed, tensor_id("prompt"), n0, sh.vocab - 1).numpy()
    t.prefill(0, prompt, k)
    sched = acceptance_schedule(SCHEDULE_SEED, steps + warmup, k).numpy()
    for i in range(warmup):
        t.step_async([0], [int(sched[i])]); t.step_wait()
    n_start = t.seq_len(0)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    a.record(stream)
    tokens = pipelined_steps(t, [0], [[int(sched[warmup + i])] for i in range(steps)])
    b.record(stream)
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / steps
    n_mid = (n_start + t.seq_len(0)) // 2
    cls, _ = measure_classes(t, [0], [8], impl)
    t.close()
    pk, pk_src = peaks()
    cost = step_cost(sh, k, n_mid)
    t_hbm = cost["bytes"] / (pk["hbm_gbs"] * 1e9) * 1e3
    t_tensor = cost["flops"] / (pk["bf16_tflops_sustained"] * 1e12) * 1e3
    gemm_ms = cls.get("gemm", 0.0) + cls.get("lmhead", 0.0)
    return {"config": workload_config(sh, k, n0, 1), "steps": steps, "warmup": warmup, "ms_per_step": ms, "tokens_per_s": tokens / (ms * steps) * 1e3,
            "mean_accept_len": tokens / steps,
            "step_roofline": {"bytes": cost["bytes"], "flops": cost["flops"], "n_cached": n_mid, "t_hbm_ms": t_hbm, "t_tensor_ms": t_tensor,
                              "frac_measured_peaks": max(t_hbm, t_tensor) / ms,
                              "frac_nominal_peaks": max(cost["bytes"] / (NOMINAL["hbm_gbs"] * 1e9), cost["flops"] / (NOMINAL["bf16_tflops"] * 1e12)) * 1e3 / ms,
                              "peak_source": pk_src},
            "roofline": {"bound": "tensor" if t_tensor >= t_hbm else "hbm",
                         "achieved": (cost["gemm_flops"] / (gemm_ms * 1e-3) / 1e12) if t_tensor >= t_hbm else (cost["weight_bytes"] / (gemm_ms * 1e-3) / 1e9),
                         "peak": pk["bf16_tflops_sustained"] if t_tensor >= t_hbm else pk["hbm_gbs"], "unit": "TFLOP/s" if t_tensor >= t_hbm else "GB/s",
                         "frac": ((cost["gemm_flops"] / (gemm_ms * 1e-3) / 1e12) / pk["bf16_tflops_sustained"]) if t_tensor >= t_hbm
                                 else ((cost["weight_bytes"] / (gemm_ms * 1e-3) / 1e9) / pk["hbm_gbs"]),
                         "launch_ms_per_step": round(gemm_ms, 4), "class_ms_per_step": {x: round(y, 4) for x, y in cls.items()}}}


def prefill_bench(sh, impl, dev, n_prompts=(1024, 4096), reps=3):
    """First-pass (prompt encoding) time: the default chunks of one decode step's rows against one
    pass per prompt (`prefill_rows`), one JSON line per case.  A diagnostic beside the step benchmark."""
    from paper_2511_08923_b200 import Tidar, pack_weights
    pk, _ = peaks()
    packed = pack_weights(gen_model_weights(sh, device=dev), dev)
    k = sh.k
    per_layer = (sh.d_model * (sh.n_q_heads + 2 * sh.n_kv_heads) * sh.head_dim + sh.n_q_heads * sh.head_dim * sh.d_model + 3 * sh.d_model * sh.d_ffn)
    for n in n_prompts:
        prompt = gen_token_ids(sh.seed, tensor_id("prompt"), n, sh.vocab - 1).numpy()
        for rows in (0, n + k):
            t = Tidar(sh, packed, k_max=k, max_batch=1, max_seq_len=n + 4 * k + 64, impl=impl, device=dev, prefill_rows=rows)
            t.prefill(0, prompt, k)
            torch.cuda.synchronize()
            w0 = time.perf_counter()
            for _ in range(reps):
                t.prefill(0, prompt, k)
            torch.cuda.synchronize()
            ms = (time.perf_counter() - w0) / reps * 1e3
            flops = 2.0 * (n + k) * sh.n_layers * per_layer + sum(4.0 * sh.n_q_heads * sh.head_dim * (g + 1) for g in range(n)) * sh.n_layers
            print(json.dumps({"prefill_bench": {"workload": sh.name, "prompt_len": n, "k": k, "prefill_rows": rows or "default (rows of a decode step)"},
                              "ms": round(ms, 2), "prompt_tokens_per_s": round(n / ms * 1e3, 1), "tflops": round(flops / ms / 1e9, 1),
                              "frac_of_measured_bf16_peak": round(flops / ms / 1e9 / pk["bf16_tflops_sustained"], 3)}))
            t.close()


def workload_config(sh, k, n0, batch):
    return {"workload": f"TiDAR decode step, {sh.name}-class decoder ({sh.n_layers} layers, d_model {sh.d_model}, "
                        f"{sh.n_q_heads}/{sh.n_kv_heads} heads, head_dim {sh.head_dim}, ffn {sh.d_ffn}, vocab {sh.vocab}), "
                        f"bf16 random-init seed {sh.seed}, batch {batch}, prompt {n0} random ids, k={k} ({k*(k+1)} slots/step), greedy",
            "acceptance": f"seeded truncated-geometric schedule (seed {SCHEDULE_SEED}, p=0.8969, mean 8 at k=16)",
            "l2": "inputs larger than L2: each step streams every weight once (>> 126 MB)",
            "k": k, "prompt_len": n0, "batch": batch}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=128)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="8b", choices=list(CONFIGS))
    ap.add_argument("--kernels", type=int, default=None, help="library impl: 0 tensor-core, 1 replay (diagnostic)")
    ap.add_argument("--layers", type=int, default=None, help="reduced-depth twin (diagnostics only; not a bench value)")
    ap.add_argument("--k", type=int, default=None)
    ap.add_argument("--batch", type=int, default=1, help="sequences decoded together (the batch / block sweep; default 1)")
    ap.add_argument("--prompt-len", type=int, default=None, help="cached positions per sequence at the start (default: the workload's)")
    ap.add_argument("--per-l-steps", type=int, default=2)
    ap.add_argument("--ar-steps", type=int, default=32, help="steps of the k = 1 autoregressive reference (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--ref-steps", type=int, default=1, help="whole oracle steps the reference arm / CPU baseline times (one 8B-class step is ~10 s of float64 work)")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the 1.5B-class step that the default run reports beside the 8B-class one")
    ap.add_argument("--prefill-bench", action="store_true", help="time the first pass over 1 k and 4 k prompts, default chunks against one pass, and exit")
    ap.add_argument("--attn-microbench", action="store_true", help="time the attention entry point alone at 1 k .. 32 k cached positions and exit")
    ap.add_argument("--lib-debug", type=int, default=0, help="library debug bits (4: bf16 split-K partial sums, 8: plain launches instead of the graph; diagnostics, not the bench configuration)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    sh = CONFIGS[args.workload]
    if args.layers:
        sh = sh.reduced(args.layers)
    k = args.k or sh.k
    n0 = args.prompt_len or sh.prompt_len
    B = args.batch
    if args.impl == "reference":
        run_reference(args, sh, k, n0)
        return

    if args.attn_microbench:
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
        attention_microbench()
        return
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path); use --impl reference for the oracle")
    if args.prefill_bench:
        prefill_bench(sh, args.kernels if args.kernels is not None else DEFAULT_IMPL, "cuda:0")
        return
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = f"cuda:{local}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev))

    from paper_2511_08923_b200 import Tidar, pack_weights
    impl = args.kernels if args.kernels is not None else DEFAULT_IMPL
    wt = gen_model_weights(sh, device=dev)
    packed = pack_weights(wt, dev)
    del wt
    torch.cuda.empty_cache()
    stream = torch.cuda.Stream(device=dev)
    n_steps_total = args.warmup + 2 * args.steps + 8 + k * args.per_l_steps
    t = Tidar(sh, packed, k_max=k, max_batch=B, max_seq_len=n0 + (n_steps_total + 4) * k + 2 * k + 64, impl=impl,
              device=dev, stream=stream, debug=args.lib_debug)
    prompt = gen_token_ids(sh.seed, tensor_id("prompt"), n0, sh.vocab - 1).numpy()
    seqs = list(range(B))
    for b in seqs:
        t.prefill(b, np.roll(prompt, b), k)
    sched = acceptance_schedule(SCHEDULE_SEED, args.warmup + 2 * args.steps + B, k).numpy()

    def forced(si, L=None):           # sequence b of step si takes the schedule's entry si + b
        return [int(sched[si + b]) if L is None else L for b in seqs]

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K steps, CUDA events on the library's stream -----
    si = 0
    for _ in range(args.warmup):
        t.step_async(seqs, forced(si)); t.step_wait(); si += 1
    n_start = t.seq_len(0)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = t.launch_count()
    barrier()
    with ClockSampler(local) as clk:
        with torch.cuda.stream(stream):
            ev0.record(stream)
        tokens = pipelined_steps(t, seqs, [forced(si + j) for j in range(args.steps)]); si += args.steps
        with torch.cuda.stream(stream):
            ev1.record(stream)
        barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = t.launch_count() - launches0
    n_mid = (n_start + t.seq_len(0)) // 2
    clocks = clk.summary()

    # ---- end to end through tidar_step with host buffers (wall clock) --------------
    barrier()
    w0 = time.perf_counter()
    # (tidar_step_async / tidar_step_wait with two steps in flight: each step's inputs go from the library's
    # pinned staging to the device and its results come back into pinned memory and out to these arrays)
    tokens_e2e = pipelined_steps(t, seqs, [forced(si + j) for j in range(args.steps)]); si += args.steps
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - w0

    # ---- per-class kernel time ----------------------------------------------------------
    # (a) in the launch mode that was just timed (replayed graph, programmatic launches): every kernel
    #     stamps the moment its first CTA got past the previous kernel and the moment its last CTA
    #     finished (tidar_debug_set_timeline); a class's time is the sum of those intervals;
    # (b) plain launches, each bracketed by CUDA events (no overlap between kernels): for comparison.
    cls, cls_plain = measure_classes(t, seqs, forced(0, 8 if k >= 8 else k), impl)

    # ---- per acceptance length -----------------------------------------------------------
    per_L = {}
    # every L starts from the same context (a fresh first pass over the prompt and one untimed
    # step), so that the latencies differ by L alone and not by how far the cache has grown
    for L in (range(1, k + 1) if args.per_l_steps > 0 else ()):
        for b_ in seqs:
            t.prefill(b_, np.roll(prompt, b_), k)
        t.step_async(seqs, forced(0, L)); t.step_wait()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        pipelined_steps(t, seqs, [forced(0, L)] * args.per_l_steps)
        b.record(stream)
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / args.per_l_steps
        per_L[str(L)] = {"ms_per_step": round(ms, 4), "tokens_per_s": round(B * L / ms * 1e3, 1)}

    # ---- autoregressive reference on the same kernels: one causal slot per pass (tidar_ar_step) ----
    # The paper's headline is decode tokens/s relative to plain AR decoding of the same model
    # (Section 4.3); this gives the same ratio on this GPU.  An AR step carries the settled token
    # alone (T = 1, no mask slots) and always emits exactly one token.
    ar = None
    if args.ar_steps > 0 and B == 1:
        t.close()
        t = Tidar(sh, packed, k_max=1, max_batch=1, max_seq_len=n0 + args.ar_steps + 16, impl=impl, device=dev, stream=stream,
                  debug=args.lib_debug)
        t.prefill(0, prompt, 1)
        for _ in range(3):
            t.ar_step([0])
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        a.record(stream)
        for _ in range(args.ar_steps):
            t.ar_step([0])
        b.record(stream)
        torch.cuda.synchronize()
        ar_ms = a.elapsed_time(b) / args.ar_steps
        ar = {"ms_per_step": round(ar_ms, 4), "tokens_per_s": round(1e3 / ar_ms, 1), "steps": args.ar_steps, "slots_per_step": 1,
              "hbm_frac_of_measured_peak": None}

    if world > 1:
        ms_total, e2e_s, tokens, tokens_e2e = aggregate_over_ranks(ms_total, e2e_s, tokens, tokens_e2e, dev)
    t.close()
    t, packed = None, None
    torch.cuda.empty_cache()

    # ---- the other model class the target names (1.5B-class, k = 16): same kernels, a short run (N = 1 only) ----
    other = None
    if world == 1 and args.workload == "8b" and not args.layers and B == 1 and args.k is None and not args.no_other_workloads:
        other = {"1.5b": measure_other_workload(CONFIGS["1.5b"], impl, dev, stream, steps=64)}

    if rank == 0:
        pk, pk_src = peaks()
        ms_step = ms_total / args.steps
        cost = step_cost(sh, k, n_mid, batch=B)
        t_hbm = cost["bytes"] / (pk["hbm_gbs"] * 1e9) * 1e3
        t_tensor = cost["flops"] / (pk["bf16_tflops_sustained"] * 1e12) * 1e3
        t_hbm_nom = cost["bytes"] / (NOMINAL["hbm_gbs"] * 1e9) * 1e3
        t_tensor_nom = cost["flops"] / (NOMINAL["bf16_tflops"] * 1e12) * 1e3
        # Dominant kernel: gemm_tc_kernel (every projection and the LM head; three epilogue
        # variants of one kernel).  Its launches of one step are timed one by one with CUDA
        # events on the library's stream (classes "gemm" and "lmhead"; the LM-head class also
        # holds the small argmax merge kernel).
        gemm_ms = cls.get("gemm", 0.0) + cls.get("lmhead", 0.0)
        n_gemm_launches = 4 * sh.n_layers + 1
        tensor_bound = t_tensor >= t_hbm
        if tensor_bound:
            ach = cost["gemm_flops"] / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
            roof = {"bound": "tensor", "achieved": ach, "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s"}
        else:
            ach = cost["weight_bytes"] / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0
            roof = {"bound": "hbm", "achieved": ach, "peak": pk["hbm_gbs"], "unit": "GB/s"}
        tr = TRAFFIC.get(args.workload) if (B == 1 and k == sh.k and not args.layers and not args.prompt_len) else None
        roof.update({"frac": roof["achieved"] / roof["peak"],
                     "traffic": tr["bytes_per_step"] if tr else None,
                     "traffic_note": tr["note"] if tr else "no ncu capture of this workload since the kernel last changed",
                     "kernel": f"gemm_tc_kernel, all {n_gemm_launches} launches of one step (QKV, O, gate/up, down per layer + LM head; the class also "
                               "holds the two small kernels that finish them: the SwiGLU fix-up of K-split tiles and the argmax merge)",
                     "algorithmic": {"flops_per_step": cost["gemm_flops"], "weight_bytes_per_step": cost["weight_bytes"]},
                     "peak_source": pk_src + (" (bf16 matmul, sustained: the kernel runs inside a long step)" if tensor_bound else " (copy bandwidth)"),
                     "launch_ms_per_step": round(gemm_ms, 4), "class_ms_per_step": {a: round(b, 4) for a, b in cls.items()},
                     "timing_mode": "in-kernel %globaltimer stamps inside the replayed graph (the mode `value` is timed in): per launch, latest CTA end "
                                    "minus earliest CTA start after its dependency; 'busy' = sum over all launches, 'span' = first start to last end",
                     "class_ms_plain_launches": {a: round(b, 4) for a, b in cls_plain.items()}})
        line = {"metric": "decode_tokens_per_s", "value": tokens / (ms_total * 1e-3), "unit": "tokens/s", "n_gpus": world,
                "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
                "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
                "config": workload_config(sh, k, n0, B), "clocks": clocks,
                "e2e": {"value": tokens_e2e / e2e_s, "unit": "tokens/s", "h2d_bytes_per_step": 8 * B, "d2h_bytes_per_step": 4 * (k + 1) * B,
                        "ms_per_step": 1e3 * e2e_s / args.steps, "api": "tidar_step_async / tidar_step_wait, two steps in flight"},
                "gpu_launches": int(launches),
                "roofline": roof,
                "step_roofline": {"bytes": cost["bytes"], "flops": cost["flops"], "n_cached": n_mid,
                                  "t_hbm_ms": t_hbm, "t_tensor_ms": t_tensor, "frac_measured_peaks": max(t_hbm, t_tensor) / ms_step,
                                  "frac_nominal_peaks": max(t_hbm_nom, t_tensor_nom) / ms_step, "peaks": pk, "peak_source": pk_src},
                "mean_accept_len": tokens / (args.steps * world * B), "per_accept_len": per_L,
                "ar_reference": ar,
                "kernels": "tcgen05" if impl == 0 else "replay (fp32 CUDA cores)",
                "paper_context": "paper reports 4.71x (1.5B) / 5.91x (8B) tokens/s over AR on one H100; no absolute figure"}
        if ar:
            ar["hbm_frac_of_measured_peak"] = round(step_cost(sh, 1, n0)["bytes"] / (pk["hbm_gbs"] * 1e9) / (ar["ms_per_step"] * 1e-3), 4)
            ar["tidar_over_ar"] = round(line["value"] / ar["tokens_per_s"], 3)
            ar["paper"] = "4.71x (1.5B) / 5.91x (8B) on one H100 with trained drafts (mean acceptance 7.45 / 8.25 tokens per pass)"
        if other is not None:
            line["other_workloads"] = other
        if not args.no_cpu_baseline and world == 1:
            step_s, gen_s = oracle_step_timed(sh, k, n0, args.ref_steps)
            mean_L = float(sched.mean())
            line["cpu_baseline"] = {"value": mean_L / step_s, "unit": "tokens/s", "cores": blas_threads(), "kind": "oracle", "extrapolated": False,
                                    "sample": f"{args.ref_steps} whole decode step(s) of the unmodified oracle (all {sh.n_layers} layers, full LM head, "
                                              f"k={k}, n={n0} cached positions), float64 NumPy, {step_s:.1f} s per step; weights handed over layer "
                                              f"by layer, their production ({gen_s:.1f} s) not counted"}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def aggregate_over_ranks(ms_total, e2e_s, tokens, tokens_e2e, device):
    """Replicas only: every rank decodes its own sequence, nothing is exchanged on the data path.
    The job's time is the slowest rank's (MAX), its tokens are all ranks' tokens (SUM).  The
    process group is the caller's (NCCL under torchrun; gloo in the CPU test)."""
    import torch.distributed as dist
    tt = torch.tensor([ms_total, e2e_s], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    tk = torch.tensor([tokens, tokens_e2e], device=device, dtype=torch.float64)
    dist.all_reduce(tk, op=dist.ReduceOp.SUM)
    return float(tt[0]), float(tt[1]), float(tk[0]), float(tk[1])


DEFAULT_IMPL = 0
# dram__bytes_read.sum + dram__bytes_write.sum of gemm_tc_kernel per step, from the ncu capture
# summarised in profiles/ (2-layer twin of the workload; per-layer traffic x n_layers + the LM
# head launch).  Removed whenever the kernel changes after the capture.
TRAFFIC = {
    "8b": {"bytes_per_step": 36 * (111.0e6 + 53.6e6 + 35.9e6 + 208.6e6) + 1252.3e6,
           "note": "ncu dram read+write per launch on the 2-layer twin (down 111.0, QKV 53.6, O 35.9, gate/up 208.6 MB; LM head "
                   "1252.3 MB), x 36 layers + LM head; see profiles/gemm_tc_kernel_8b_shapes_R272.md"},
}

if __name__ == "__main__":
    main()

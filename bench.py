#!/usr/bin/env python
"""Benchmark of the Elastic Cache hot path on B200.

One "step" is one pass of the whole path over one synthetic batch: importance over the
prompt, anchor selection + merge into the compacted cache, then the workload's full decode
loop (attention over the cache + fixed-point eviction every token). The reported value is
generated tokens per second over that whole pass, all problems of all ranks counted.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

The headline workload is the largest 7B-shaped configuration (batch 8, 1024-token prompts: a
1.07 GB compacted cache, many times the L2). At one GPU the same JSON line carries, under
`per_workload`, the other configurations (7B batch 1, the 13B keep-ratio sweep, the 8192-token
stress case) timed the same way with fewer passes, and a read-only stream rate measured in the
same process beside the copy rate the roofline fractions are quoted against.

Under torchrun every rank runs its own batch (independent problems: no data-path collective),
times on the device, and rank 0 prints one JSON line with the max-over-ranks time.
`--impl reference` times the CPU oracle (the deliberately plain fp64 program the tests check
against) on a bounded sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2407_18121_b200 import workloads as wl  # noqa: E402

METRIC = "decode tokens/s on merged KV (whole pass: importance + select/merge + decode loop)"
UNIT = "tokens/s"


HEADLINE = "llava7b_b8"
# the other configurations, reported under `per_workload` at one GPU (every keep ratio of each)
OTHER_WORKLOADS = ("llava7b_b1", "llava13b_b4", "long8k")

# DRAM bytes (read + write) of one decode_kernel launch (a later step of the loop) taken from a profiler
# capture of this benchmark on a subset of the headline workload's problems and scaled to the full
# launch by the number of units (every unit streams its own rows once: traffic is proportional to
# units); valid only for the kernel source it was taken on (sha1 prefix of csrc/ec_decode.cu),
# otherwise reported as null.
DECODE_TRAFFIC = {"source_sha1": "377b9a4c455b", "llava7b_b8": 4 * (270075904 + 3330560)}


def decode_traffic(workload: str):
    import hashlib
    path = os.path.join(ROOT, "paper_2407_18121_b200", "csrc", "ec_decode.cu")
    try:
        digest = hashlib.sha1(open(path, "rb").read()).hexdigest()
    except OSError:
        return None
    if not DECODE_TRAFFIC["source_sha1"] or not digest.startswith(DECODE_TRAFFIC["source_sha1"]):
        return None
    return DECODE_TRAFFIC.get(workload)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.rows.append(parts)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                mx.append(float(r[1]))
            except ValueError:
                continue
            for name, val in zip(names, r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def bits_to_tensor(bits: np.ndarray, pin: bool):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t.pin_memory() if pin else t


# ----------------------------------------------------------------------------- CPU oracle leg

def oracle_sample_size(w: wl.Workload, budget_fma: float = 2.0e11):
    """Picks how much of the workload the oracle is timed on: the whole pass when its
    multiply-add count fits the budget (tens of seconds on a many-core host), otherwise the
    first problems and the first decode steps, in proportion."""
    from oracle import ec_oracle as orc
    C_keep = orc.keep_count(w.prompt_len, w.keep_ratio)
    prompt = w.heads * w.prompt_len * (w.prompt_len + 1) / 2 * w.head_dim          # per problem
    decode = w.heads * (C_keep + 1) * w.head_dim * 2                              # per problem per step
    problems = int(max(1, min(w.N, (budget_fma / 2) // prompt)))
    steps = int(max(4, min(w.decode_steps, (budget_fma / 2) // (decode * problems))))
    return problems, steps


def oracle_sample(w: wl.Workload, decode_steps_sample: int = 0, problems_sample: int = 0,
                  budget_fma: float = 2.0e11):
    """Times the oracle, as it stands, on a bounded sample and scales linearly to the whole pass.
    Sample: the full prompt stage (importance, selection, buckets, merge) of the first
    `problems_sample` problems, then `decode_steps_sample` decode steps on them."""
    from oracle import ec_oracle as orc
    auto_p, auto_s = oracle_sample_size(w, budget_fma)
    problems = list(range(min(problems_sample or auto_p, w.N)))
    Qb, Kb, Vb = wl.prompt(w, problems)
    T = w.prompt_len
    C = orc.keep_count(T, w.keep_ratio)
    t0 = time.perf_counter()
    scores, _ = orc.importance(Qb, Kb, w.scale)
    anchors = orc.select(scores, C, True)
    lo, hi = orc.buckets(anchors, T)
    Kc, Vc = orc.merge(Kb, lo, hi), orc.merge(Vb, lo, hi)
    queue = orc.DecodeQueue(orc.widen_bf16(orc.round_bf16(Kc)), orc.widen_bf16(orc.round_bf16(Vc)), cap=C + 1)
    t1 = time.perf_counter()
    S = min(decode_steps_sample or auto_s, w.decode_steps)
    dec_in = [wl.decode_step_inputs(w, s, problems) for s in range(S)]
    t2 = time.perf_counter()
    for s in range(S):
        q, k, v = dec_in[s]
        queue.step(q, k, v, w.scale, policy=orc.POLICY_FIXED, budget=C, offset=w.offset)
    t3 = time.perf_counter()
    frac = w.N / len(problems)
    prompt_s = (t1 - t0) * frac
    decode_s = (t3 - t2) * frac * (w.decode_steps / S)
    total = prompt_s + decode_s
    whole = len(problems) == w.N and S == w.decode_steps
    return {"seconds_whole_pass_extrapolated": total, "prompt_s": prompt_s, "decode_s": decode_s,
            "sample_seconds": (t1 - t0) + (t3 - t2), "cores": orc.num_threads(),
            "sample": ("the whole pass (every problem, every decode step)" if whole else
                       f"prompt stage of {len(problems)} of {w.N} problems (all {w.heads} heads) + {S} of "
                       f"{w.decode_steps} decode steps on them, scaled linearly to the whole pass")}


def run_reference(args, w: wl.Workload):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import ec_oracle as orc
    per_step = []
    info = None
    # a step here is one bounded sample; its size shrinks with the number of steps asked for, so that
    # the whole run stays within a few minutes (about 0.5e10 multiply-adds per second on 16 cores)
    budget = min(2.0e11, 1.0e12 / max(1, args.warmup + args.steps))
    for i in range(args.warmup + args.steps):
        info = oracle_sample(w, args.oracle_decode_steps, args.oracle_problems, budget)
        if i >= args.warmup:
            per_step.append(info["seconds_whole_pass_extrapolated"])
    sec = float(np.mean(per_step))
    tokens = w.batch * w.decode_steps
    value = tokens / sec
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(w, orc.keep_count(w.prompt_len, w.keep_ratio)),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": info["cores"], "kind": "oracle",
                             "sample": info["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def workload_config(w: wl.Workload, n_keep: int):
    return {"workload": w.name, "batch": w.batch, "layers": w.layers, "heads": w.heads, "head_dim": w.head_dim,
            "prompt_len": w.prompt_len, "keep_ratio": w.keep_ratio, "decode_steps": w.decode_steps,
            "offset": w.offset, "population": "per_head", "protect_ends": True, "l2": l2_statement(w, n_keep)}


L2_BYTES = 126e6


def l2_statement(w: wl.Workload, n_keep: int) -> str:
    """Whether the data each timed stage streams exceeds the 126 MB L2 (nothing is flushed between passes)."""
    units = w.N * w.heads
    prompt = units * w.prompt_len * w.head_dim * 2                    # each of Q, K, V
    cache = 2 * units * n_keep * w.head_dim * 2                       # K and V rows read by every decode step
    if prompt > L2_BYTES and cache > L2_BYTES:
        return (f"inputs larger than L2 (prompt Q, K, V {prompt / 1e6:.0f} MB each and the compacted cache "
                f"{cache / 1e6:.0f} MB per step exceed 126 MB)")
    small = [n for n, b in (("prompt tensors", prompt), ("compacted cache", cache)) if b <= L2_BYTES]
    return (f"NOT larger than L2: {' and '.join(small)} fit the 126 MB L2 (prompt {prompt / 1e6:.0f} MB per tensor, "
            f"cache {cache / 1e6:.0f} MB), so the bandwidth figures of this workload are L2-assisted")



# ----------------------------------------------------------------------------- rank logic

def rank_workload(w: wl.Workload, rank: int) -> wl.Workload:
    """The batch a rank works on: same shapes, its own seed. Ranks never exchange data."""
    import dataclasses
    return dataclasses.replace(w, seed=w.seed + 1000 * rank)


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return [float(x) for x in values]
    t = torch.tensor(values, dtype=torch.float64, device=device or "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_tokens_per_s(w: wl.Workload, world: int, ms_per_pass: float) -> float:
    """Every rank generates batch * decode_steps tokens per pass; the job's time is the slowest rank's."""
    return w.batch * w.decode_steps * world / (ms_per_pass * 1e-3)


# ----------------------------------------------------------------------------- GPU leg

def stage_figures(w: wl.Workload, C: int, imp_ms: float, mrg_ms: float, dec_ms: float, peaks: dict):
    """Algorithmic work of the three stages of one pass and the rates the measured times give."""
    units, T, D, S = w.N * w.heads, w.prompt_len, w.head_dim, w.decode_steps
    w_ratio = w.keep_ratio
    # one decode launch: every cached K and V row once, q/k_new/v_new in, out and the overwritten slot out
    dec_bytes = units * (2 * C * D * 2 + 3 * D * 2 + D * 2 + 2 * D * 2)
    dec_gbs = dec_bytes / (dec_ms * 1e-3 / S) / 1e9
    # select + merge: K, V and scores in, kept rows and the index map out
    mrg_bytes = units * (2 * T * D * 2 + 4 * T + 2 * C * D * 2 + 4 * C)
    mrg_gbs = mrg_bytes / (mrg_ms * 1e-3) / 1e9
    # two passes, each 2*D flops for the T(T+1)/2 causal scores
    imp_flops = 2.0 * D * T * (T + 1) * units
    imp_tflops = imp_flops / (imp_ms * 1e-3) / 1e12

    def hbm(gbs):
        return {"achieved": gbs, "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                "frac_of_read_stream": (gbs / peaks["read_gbs"]) if peaks.get("read_gbs") else None,
                "frac_of_nominal_8TBs": gbs / 8000.0}

    dec = hbm(dec_gbs)
    dec["bytes_per_launch"] = dec_bytes
    mrg = hbm(mrg_gbs)
    mrg["bytes_per_call"] = mrg_bytes
    mixed, w = mixed_peak_for(peaks, w_ratio)
    mrg["frac_of_mixed_stream"] = (mrg_gbs / mixed) if mixed else None
    mrg["mixed_stream_peak"] = mixed
    mrg["mixed_stream_write_every"] = w
    imp = {"achieved": imp_tflops, "unit": "TFLOP/s", "frac": imp_tflops / peaks["bf16_tflops"],
           "flops_per_call": imp_flops}
    return dec, mrg, imp


class DevicePass:
    """One workload resident on the device and the three calls of a pass over it."""

    def __init__(self, w: wl.Workload, host=None, resident=None):
        """`host`: six host tensors (Q, K, V, q, k, v) to upload; or `resident`: another DevicePass whose
        device inputs are reused (a further keep ratio over the same prompt)."""
        from paper_2407_18121_b200 import binding as ec
        from paper_2407_18121_b200.session import ElasticCacheSession
        import torch
        self.ec, self.w = ec, w
        if resident is not None:
            self.Q, self.K, self.V, self.q, self.k, self.v, self.out = (resident.Q, resident.K, resident.V, resident.q,
                                                                      resident.k, resident.v, resident.out)
        else:
            self.Q, self.K, self.V, self.q, self.k, self.v = (t.cuda() for t in host)
            self.out = torch.empty_like(self.q)
        self.sess = ElasticCacheSession(w.N, w.heads, w.prompt_len, w.head_dim, w.keep_ratio, w.offset, w.scale)
        self.C = self.sess.n_keep
        self.stream = torch.cuda.current_stream()

    def run(self, events=None):
        ec, sess, w = self.ec, self.sess, self.w
        if events is not None:
            events[0].record(self.stream)
        ec.ec_importance(self.Q, self.K, sess.scores, None, sess.scale, sess.ws_imp)
        if events is not None:
            events[1].record(self.stream)
        ec.ec_select_merge(self.K, self.V, sess.scores, self.C, sess.population, True, sess.Kc, sess.Vc,
                           sess.anchor_pos, None, sess.ws_sel)
        sess.cache = ec.ec_cache_init(sess.Kc, sess.Vc, self.C, self.C, w.offset)
        if events is not None:
            events[2].record(self.stream)
        sess.decode(self.q, self.k, self.v, self.out)
        if events is not None:
            events[3].record(self.stream)

    def timed(self, warmup: int, steps: int, barrier, sampler, min_ms: float = 0.0):
        """`warmup` untimed passes, then `steps` timed ones (more when `min_ms` asks for a longer timed
        region, so that the clock sampler sees it): whole time from one event pair around all of them,
        stage times as means of per-pass event pairs. Returns (ms_per_pass, imp, mrg, dec, clocks, steps)."""
        import torch
        w0, w1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        for i in range(warmup):
            if i == warmup - 1:
                w0.record(self.stream)
            self.run()
        w1.record(self.stream)
        barrier()
        if min_ms > 0.0 and warmup > 0:
            steps = max(steps, int(np.ceil(min_ms / max(w0.elapsed_time(w1), 1e-3))))
        if sampler is not None:
            sampler.start()
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(4)] for _ in range(steps)]
        t_begin, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_begin.record(self.stream)
        for i in range(steps):
            self.run(ev[i])
        t_end.record(self.stream)
        barrier()
        clocks = sampler.stop() if sampler is not None else None
        status = self.ec.ec_device_status(self.sess.ws_imp)
        if status != self.ec.EC_OK:
            raise SystemExit(f"device status {status}: {self.ec.status_string(status)}")
        return (t_begin.elapsed_time(t_end) / steps,
                float(np.mean([e[0].elapsed_time(e[1]) for e in ev])),
                float(np.mean([e[1].elapsed_time(e[2]) for e in ev])),
                float(np.mean([e[2].elapsed_time(e[3]) for e in ev])), clocks, steps)


def host_inputs(w: wl.Workload, pin: bool, threads: int):
    Qb, Kb, Vb = wl.prompt(w, threads=threads)
    qb, kb, vb = wl.decode_inputs(w, threads=threads)
    return tuple(bits_to_tensor(x, pin) for x in (Qb, Kb, Vb, qb, kb, vb))


def stream_peaks(ec, nbytes: int = 4 << 30, reps: int = 5):
    """Streaming rates of this GPU, measured here and now with the library's probe kernel over a 4 GiB
    buffer (far above the L2), best of `reps`, CUDA-event timed: read-only, and reads with one 256-byte
    row in 2 / 4 / 10 written back (the mixes of a merge at keep ratio 0.5 / 0.25 / 0.1; bytes counted
    are reads + writes). Returns {"read_gbs": ..., "mixed_gbs": {2: ..., 4: ..., 10: ...}}."""
    import torch
    buf = torch.empty(nbytes, dtype=torch.uint8, device="cuda")
    buf.zero_()
    dst = torch.empty(nbytes // 2, dtype=torch.uint8, device="cuda")
    sink = torch.zeros(1, dtype=torch.int32, device="cuda")
    stream = torch.cuda.current_stream()

    def best_of(w):
        run = (lambda: ec.ec_probe_read_stream(buf, sink)) if w == 0 else (lambda: ec.ec_probe_mixed_stream(buf, dst, w, sink))
        run()
        torch.cuda.synchronize()
        best = None
        for _ in range(reps):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            run()
            b.record(stream)
            torch.cuda.synchronize()
            ms = a.elapsed_time(b)
            best = ms if best is None else min(best, ms)
        moved = nbytes + (nbytes // w if w else 0)
        return moved / (best * 1e-3) / 1e9

    out = {"read_gbs": best_of(0), "mixed_gbs": {w: best_of(w) for w in (2, 4, 10)}}
    del buf, dst
    torch.cuda.empty_cache()
    return out


def mixed_peak_for(peaks: dict, keep_ratio: float):
    """The measured mixed-stream rate whose write share is nearest to a merge at this keep ratio."""
    mixed = peaks.get("mixed_gbs")
    if not mixed:
        return None, None
    w = min(mixed, key=lambda k: abs(1.0 / k - keep_ratio))
    return mixed[w], w


def measure_other_workloads(ec, peaks, threads: int, passes: int, local: int):
    """The remaining configurations, each timed like the headline (same calls, same event placement)
    with 3 warm-up and at least `passes` timed passes (at least 0.4 s of them); every keep ratio of a sweep is its own entry."""
    import dataclasses
    import gc
    import torch
    result = {}
    for name in OTHER_WORKLOADS:
        base = wl.WORKLOADS[name]
        host = host_inputs(base, False, threads)
        first = None
        for ratio in base.keep_ratios:
            w = dataclasses.replace(base, keep_ratios=(ratio,))
            dp = DevicePass(w, host=host) if first is None else DevicePass(w, resident=first)
            first = first or dp
            ms, imp_ms, mrg_ms, dec_ms, clocks, done = dp.timed(3, passes, torch.cuda.synchronize, ClockSampler(local),
                                                                min_ms=400.0)
            dec, mrg, imp = stage_figures(w, dp.C, imp_ms, mrg_ms, dec_ms, peaks)
            key = name if len(base.keep_ratios) == 1 else f"{name}@{ratio:g}"
            result[key] = {
                "config": workload_config(w, dp.C), "passes": done, "ms_per_pass": ms,
                "tokens_per_s": w.batch * w.decode_steps / (ms * 1e-3),
                "stages_ms": {"importance": imp_ms, "select_merge": mrg_ms, "decode_loop": dec_ms,
                              "decode_per_token_us": dec_ms * 1e3 / w.decode_steps},
                "decode_splits": ec.ec_decode_splits(dp.sess.cache),
                "decode": dec, "merge": mrg, "importance": imp, "clocks": clocks}
            if dp is not first:
                del dp.sess
        del first, dp, host
        gc.collect()
        torch.cuda.empty_cache()
    return result


def run_ours(args, w: wl.Workload):
    import torch
    import torch.distributed as dist

    from paper_2407_18121_b200 import binding as ec
    from paper_2407_18121_b200 import build as ecbuild
    from paper_2407_18121_b200.session import ElasticCacheSession

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the CUDA library is the only implementation")
    torch.cuda.set_device(local)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        ecbuild.build()
    if world > 1:
        dist.barrier()
    ec.lib()
    threads = max(1, min(16, (os.cpu_count() or 8) // max(1, world)))

    # every rank holds its own batch of independent problems (weak scaling, no exchange)
    wr = rank_workload(w, rank)
    N, H, T, D, S = wr.N, wr.heads, wr.prompt_len, wr.head_dim, wr.decode_steps
    host = host_inputs(wr, True, threads)
    Qh, Kh, Vh, qh, kh, vh = host
    dp = DevicePass(wr, host=host)
    C = dp.C
    stream = dp.stream

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    total_ms, imp_ms, mrg_ms, dec_ms, clocks, _ = dp.timed(args.warmup, args.steps, barrier,
                                                           ClockSampler(local) if rank == 0 else None)
    ms_per_step = total_ms
    splits = ec.ec_decode_splits(dp.sess.cache)

    # the same pass recorded once in a CUDA graph and replayed (reported beside the plain launches)
    graph_ms = None
    if not args.no_graph:
        side = torch.cuda.Stream()
        side.wait_stream(stream)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                dp.run()
        stream.wait_stream(side)
        for _ in range(2):
            g.replay()
        barrier()
        g0 = torch.cuda.Event(enable_timing=True)
        g1 = torch.cuda.Event(enable_timing=True)
        reps = max(1, min(args.steps, 10))
        g0.record(stream)
        for _ in range(reps):
            g.replay()
        g1.record(stream)
        barrier()
        graph_ms = g0.elapsed_time(g1) / reps
        del g

    # The fused form of the prompt stage (attention output + importance in one call: three contractions
    # instead of the two of ec_importance plus the two of an attention kernel), timed on the same
    # tensors beside the pass; it is not part of the timed pass, whose importance call is ec_importance.
    attn = None
    if not args.no_attention:
        attn_out = torch.empty_like(dp.Q)
        attn_scores = torch.empty_like(dp.sess.scores)

        def attn_call(with_scores):
            ec.ec_prefill_attention(dp.Q, dp.K, dp.V, attn_out, None, attn_scores if with_scores else None, wr.scale,
                                    dp.sess.ws_imp)

        attn_ms = {}
        for with_scores in (False, True):
            for _ in range(3):
                attn_call(with_scores)
            barrier()
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            reps = max(3, min(args.steps, 10))
            a0.record(stream)
            for _ in range(reps):
                attn_call(with_scores)
            a1.record(stream)
            barrier()
            attn_ms[with_scores] = a0.elapsed_time(a1) / reps
        if ec.ec_device_status(dp.sess.ws_imp) != ec.EC_OK:
            raise SystemExit("device status after ec_prefill_attention")
        one = 1.0 * D * T * (T + 1) * N * H                        # flops of one causal contraction
        attn = {"attention_ms": attn_ms[False], "attention_tflops": 2 * one / (attn_ms[False] * 1e-3) / 1e12,
                "attention_and_importance_ms": attn_ms[True],
                "attention_and_importance_tflops": 3 * one / (attn_ms[True] * 1e-3) / 1e12,
                "note": ("ec_prefill_attention without / with the column-sum pass; flops = 2*D per visible "
                         "(query, key) pair and contraction: two contractions for the attention, three with the importance")}
        del attn_out, attn_scores

    # end to end: inputs start in pinned host memory, results are read back every pass. Two passes are
    # in flight, each with its own session, stream and host result buffers, so that the upload of the
    # next pass's prompt overlaps the decode loop of this one (a serving loop with double buffering);
    # every copy of every pass lies inside the timed region.
    lanes = []
    for _ in range(2):
        lane_sess = ElasticCacheSession(N, H, T, D, wr.keep_ratio, wr.offset, wr.scale)
        lanes.append((lane_sess, torch.cuda.Stream(), torch.empty(qh.shape, dtype=torch.bfloat16).pin_memory(),
                      torch.empty((N, H, C), dtype=torch.int32).pin_memory()))

    def e2e_pass(i):
        lane_sess, lane_stream, lane_out, lane_anchors = lanes[i % 2]
        with torch.cuda.stream(lane_stream):
            a = lane_sess.compress_host(Qh, Kh, Vh, lane_anchors)
            b, c = lane_sess.decode_host(qh, kh, vh, lane_out)
        return a + b, c + lane_anchors.numel() * 4

    def fork():
        for _, lane_stream, _, _ in lanes:
            lane_stream.wait_stream(stream)

    def join():
        for _, lane_stream, _, _ in lanes:
            stream.wait_stream(lane_stream)

    fork()
    for i in range(2):
        e2e_pass(i)
    join()
    barrier()
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    e2e_steps = max(2, min(args.steps, 6))
    e0.record(stream)
    fork()
    for i in range(e2e_steps):
        h2d, d2h = e2e_pass(i)
    join()
    e1.record(stream)
    barrier()
    e2e_ms = e0.elapsed_time(e1) / e2e_steps
    del lanes

    ms_per_step, e2e_ms, dec_ms, mrg_ms, imp_ms = max_over_ranks([ms_per_step, e2e_ms, dec_ms, mrg_ms, imp_ms], "cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    if world == 1 and not args.no_read_peak:
        peaks.update(stream_peaks(ec))
    tokens = w.batch * S * world
    value = whole_job_tokens_per_s(w, world, ms_per_step)
    dec, mrg, imp = stage_figures(w, C, imp_ms, mrg_ms, dec_ms, peaks)
    # kernels per pass: two importance passes, selection, merge, and one decode kernel per token
    launches_per_pass = 2 + 2 + S

    roofline = {"kernel": "decode_kernel", "bound": "hbm", "achieved": dec["achieved"], "peak": peaks["hbm_gbs"],
                "unit": "GB/s", "frac": dec["frac"], "peak_source": peaks["source"] + " (copy: half reads, half writes)",
                "read_stream_peak": peaks.get("read_gbs"), "mixed_stream_peaks": peaks.get("mixed_gbs"), "frac_of_read_stream": dec["frac_of_read_stream"],
                "frac_of_nominal_8TBs": dec["frac_of_nominal_8TBs"], "bytes_per_launch": dec["bytes_per_launch"],
                "decode_splits": splits, "traffic": decode_traffic(w.name),
                "note": ("algorithmic bytes of one step / (decode loop time / steps); consecutive steps of the "
                         "loop overlap (a step reads the rows no step writes while earlier steps are in "
                         "flight), so a launch is not timed alone. `peak` is the driver-measured copy rate; "
                         "`read_stream_peak` is a read-only 16-byte-load sum over 4 GiB timed in this process")}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "storage_dtype": "bf16", "data": "synthetic",
        "config": workload_config(w, ec.ec_keep_count(w.prompt_len, w.keep_ratio)),
        "stages_ms": {"importance": imp_ms, "select_merge": mrg_ms, "decode_loop": dec_ms,
                      "decode_per_token_us": dec_ms * 1e3 / S, "whole_pass_cuda_graph_replay": graph_ms},
        "decode_only_tokens_per_s": w.batch * S * world / (dec_ms * 1e-3),
        "roofline": roofline,
        "merge": dict(mrg, note="whole ec_select_merge call (selection + merge kernels)"),
        "importance": imp,
        "prefill_attention": attn,
        "e2e": {"value": tokens / (e2e_ms * 1e-3), "unit": UNIT, "ms_per_step": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "pipeline": "two passes in flight: the next pass's prompt upload overlaps this pass's decode loop"},
        "gpu_launches": launches_per_pass * args.steps,
        "clocks": clocks,
    }
    # free the headline's tensors before the other configurations come in
    del dp, host, Qh, Kh, Vh, qh, kh, vh
    import gc
    gc.collect()
    torch.cuda.empty_cache()
    if world == 1 and not args.no_per_workload:
        line["per_workload"] = measure_other_workloads(ec, peaks, threads, args.per_workload_passes, local)
    if world == 1 and not args.no_cpu_baseline:
        o = oracle_sample(w, args.oracle_decode_steps, args.oracle_problems)
        line["cpu_baseline"] = {"value": w.batch * S / o["seconds_whole_pass_extrapolated"], "unit": UNIT,
                                "cores": o["cores"], "kind": "oracle", "sample": o["sample"],
                                "sample_seconds": o["sample_seconds"]}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=HEADLINE, choices=list(wl.WORKLOADS))
    ap.add_argument("--decode-steps", type=int, default=None, help="override the workload's decode length")
    ap.add_argument("--problems", type=int, default=None,
                    help="run only the first K problems (batch x layer pairs) of the workload: for profiling captures")
    ap.add_argument("--oracle-decode-steps", type=int, default=0)
    ap.add_argument("--oracle-problems", type=int, default=0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="skip the CUDA-graph replay measurement")
    ap.add_argument("--no-per-workload", action="store_true", help="skip the other configurations")
    ap.add_argument("--no-attention", action="store_true", help="skip the timing of ec_prefill_attention")
    ap.add_argument("--no-read-peak", action="store_true", help="skip the read-only stream measurement")
    ap.add_argument("--per-workload-passes", type=int, default=4)
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours" and not args.problems:
        args.warmup = 3                                     # timing rule: at least three warm-up passes
    w = wl.WORKLOADS[args.workload]
    if args.decode_steps:
        w = w.shrunk(decode_steps=args.decode_steps)
    if args.problems:
        w = w.shrunk(batch=1, layers=min(args.problems, w.N))      # problem n keeps its own draws
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Stream frames/s of the 24-layer compressed-KV attention path on B200.

One step = one frame (1374 tokens) through all 24 layers: append, score, evict,
quantise/pack, attention over the packed cache, via xkv_stream_step.  Prints one
JSON line (rank 0).  `--impl reference` times the CPU oracle instead.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl xkv|reference]
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
sys.path.insert(0, ROOT)

# Workload: the full stack (24 layers, 16 x 64, 1374 tokens/frame, budget 16384, 4-bit).
WORKLOAD = dict(name="full_stack_24L_1374tok_budget16384_int4", layers=24, n_heads=16, head_dim=64,
                n_tokens=1374, budget=16384, kv_bits=4, n_special=5, pool_g=16, quant_group=64, seed=3)
METRIC = "stream frames/s (24-layer compressed-KV attention)"
UNIT = "frames/s"
# dram__bytes_read.sum + dram__bytes_write.sum of one attention launch, from the ncu capture
# summarised under profiles/ (None until a capture of the current kernel exists).
ATTN_DRAM_TRAFFIC_BYTES = 23.3e6


def _peaks() -> dict:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], tflops_burst=d["bf16_tflops"], tflops_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, tflops_burst=1590.0, tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([f.strip() for f in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()
            self.thread.join(timeout=2)

    def summary(self) -> dict:
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, v in zip(names, r[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=float(np.median(sm)) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


# --------------------------------------------------------------------------- CPU oracle arm
def _oracle_layer_steps(w: dict, n_timed: int, n_warm: int):
    """Streams ONE layer through the oracle to steady state, then times whole layer-steps."""
    from oracle import xkv_oracle as xo
    from paper_2601_01204_b200 import synth
    p = xo.OracleParams(n_heads=w["n_heads"], head_dim=w["head_dim"], n_special=w["n_special"], pool_g=w["pool_g"],
                        quant_group=w["quant_group"], kv_bits=w["kv_bits"], budget=w["budget"])
    layer = xo.OracleLayer(p)
    n = w["n_tokens"]
    fill = -(-w["budget"] // n)                      # frames until the cache is full and evicting
    times = []
    for t in range(fill + n_warm + n_timed):
        q, k, v = (synth.bf16_bits_to_f32(a) for a in synth.gen_frame(w["seed"], 0, t, w["n_heads"], n, w["head_dim"]))
        t0 = time.perf_counter()
        layer.append(k, v)
        layer.score_evict(q)
        layer.quant_pack()
        if t >= fill:                                  # attention is skipped while filling (untimed)
            layer.attend(q)
        dt = time.perf_counter() - t0
        if t >= fill + n_warm:
            times.append(dt)
    return times


def _cpu_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([i.get("num_threads", 1) for i in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(w: dict, n_timed: int = 3, n_warm: int = 1) -> dict:
    times = _oracle_layer_steps(w, n_timed, n_warm)
    per_layer = float(np.mean(times))
    return dict(value=1.0 / (per_layer * w["layers"]), unit=UNIT, cores=_cpu_threads(), kind="oracle",
                sample=f"{n_timed} steady-state layer-steps of one layer (cache full at {w['budget']} tokens) timed in "
                       f"full, x{w['layers']} layers extrapolated; {per_layer:.2f} s per layer-step")


def run_reference(args) -> None:
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = WORKLOAD
    # one "step" is a bounded sample of the frame: one of the 24 (identical-shape) layer-steps
    steps, warm = max(1, min(args.steps, 12)), max(0, min(args.warmup, 2))
    t_all = time.perf_counter()
    times = _oracle_layer_steps(w, steps, warm)
    per_layer = float(np.mean(times))
    value = 1.0 / (per_layer * w["layers"])
    line = dict(impl="reference", metric=METRIC, value=value, unit=UNIT, n_gpus=args.gpus, steps=steps,
                warmup=warm, steps_requested=args.steps, warmup_requested=args.warmup, ms_per_step=per_layer * w["layers"] * 1e3, higher_is_better=True, scaling="weak",
                vs_baseline=None, dtype="f32/f64", data="synthetic",
                config=dict(workload=w["name"], layers=w["layers"], tokens_per_frame=w["n_tokens"],
                            budget=w["budget"], kv_bits=w["kv_bits"],
                            sampled_steps=steps, note="each timed step is one oracle layer-step (1/24 of a frame) "
                            "in steady state; frame time = 24 x mean"),
                cpu_baseline=dict(value=value, unit=UNIT, kind="oracle", cores=_cpu_threads(),
                                  sample=f"{steps} layer-steps, {time.perf_counter() - t_all:.0f} s total"),
                e2e=dict(value=value, unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------- GPU arm
def replica_seed(base_seed: int, rank: int) -> int:
    """Replicas stream different data: rank r uses seed base + 1000 r."""
    return base_seed + 1000 * rank


def max_over_ranks(value: float, device: str = "cuda") -> float:
    """Slowest rank's time (the replicas share nothing; the job is as slow as its slowest stream)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    tt = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def aggregate_frames_per_s(world: int, steps: int, ms_total_max: float) -> float:
    """Whole-job throughput of `world` independent replicas that each ran `steps` frames."""
    return world * steps / (ms_total_max * 1e-3)


def run_xkv(args) -> None:
    import torch
    import torch.distributed as dist
    from paper_2601_01204_b200 import build, synth
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    import paper_2601_01204_b200.xkv as xkv

    w = dict(WORKLOAD)
    if args.layers > 0:
        w["layers"] = args.layers
        w["name"] += f"_reduced_to_{args.layers}_layers"
    if args.bits == 8:
        args.keys = "once"
    w["key_mode"] = 1 if args.keys == "once" else 0
    if args.keys == "once":
        w["name"] += "_keys_once"
    if args.budget > 0 or args.bits > 0 or args.tokens > 0:      # the ablation sweep and the long-stream shape
        w["budget"] = args.budget or w["budget"]
        w["kv_bits"] = args.bits or w["kv_bits"]
        w["n_tokens"] = args.tokens or w["n_tokens"]
        w["name"] = f"stack_{w['layers']}L_{w['n_tokens']}tok_budget{w['budget']}_{ {4: 'int4', 8: 'int8', 16: 'bf16'}[w['kv_bits']] }"
        if args.keys == "once":
            w["name"] += "_keys_once"
    L, H, d, n = w["layers"], w["n_heads"], w["head_dim"], w["n_tokens"]
    p = xkv.Params(n_heads=H, head_dim=d, n_special=w["n_special"], pool_g=w["pool_g"], quant_group=w["quant_group"],
                   kv_bits=w["kv_bits"], budget=w["budget"], max_frame_tokens=n, key_mode=w["key_mode"])
    caches = [xkv.Cache(p, device=f"cuda:{local}") for _ in range(L)]
    if args.tail:
        for c in caches:
            c.xkv_set_unquantised_tail(True)
    K, W = args.steps, args.warmup
    fill = -(-w["budget"] // n)                     # 12 frames until every layer's cache is full
    pool = min(fill + W + K, 40)                    # distinct resident frames, cycled afterwards
    seed = replica_seed(w["seed"], rank)
    frames = []
    for f in range(pool):
        q = torch.empty(L, H, n, d, dtype=torch.bfloat16, device="cuda")
        k = torch.empty_like(q)
        v = torch.empty_like(q)
        for l in range(L):
            xkv.xkv_synth_fill(q[l], seed + l, l, f, synth.TENSOR_Q)
            xkv.xkv_synth_fill(k[l], seed + l, l, f, synth.TENSOR_K)
            xkv.xkv_synth_fill(v[l], seed + l, l, f, synth.TENSOR_V)
        frames.append(tuple([x[l] for l in range(L)] for x in (q, k, v)))
    out = torch.empty(L, H, n, d, dtype=torch.bfloat16, device="cuda")
    outs = [out[l] for l in range(L)]

    def step(t: int) -> None:
        q, k, v = frames[t % pool]
        xkv.xkv_stream_step(caches, q, k, v, outs)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    t = 0
    for _ in range(fill + W):                       # untimed: fill to steady state, then W warm-up steps
        step(t); t += 1
    launches0 = sum(c.xkv_get_info().launches for c in caches)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    with ClockSampler(local) as clocks:
        ev0.record()
        for _ in range(K):
            step(t); t += 1
        ev1.record()
        barrier()
    ms_total = ev0.elapsed_time(ev1)
    launches = sum(c.xkv_get_info().launches for c in caches) - launches0
    ms_total = max_over_ranks(ms_total)
    assert all(c.xkv_get_info().T == w["budget"] for c in caches)
    assert all(c.xkv_poll_status() == 0 for c in caches)

    # per-kernel device time over the same K steps, events on the launching stream
    def read_profiles() -> dict:
        acc = {}
        for c in caches:
            for name, (ms, cnt) in c.xkv_profile_read().items():
                a = acc.setdefault(name, [0.0, 0])
                a[0] += ms; a[1] += cnt
        return acc

    for c in caches:
        c.xkv_profile_enable(True)
    for _ in range(K):
        step(t); t += 1
    prof = read_profiles()
    # the same frames through the per-call entry points (one launch per call, nothing overlapped),
    # and the head-mean kernel alone: the stream step runs it beside the attention, where an
    # event pair around it also spans the time it waits for multiprocessors
    Kc = max(1, min(K, 5))
    for _ in range(Kc):
        q, k, v = frames[t % pool]; t += 1
        for l, c in enumerate(caches):
            c.kv_append(k[l], v[l]); c.kv_score_evict(q[l]); c.kv_quant_pack(); c.attn_packed_causal(q[l], outs[l])
    calls = read_profiles()
    for c in caches:
        c.xkv_debug_head_means()
    kbar_alone = read_profiles()["kbar"]
    for c in caches:
        c.xkv_profile_enable(False)

    # end to end: host tensors in pinned memory, copies inside the timed region
    Ke = max(1, min(K, 10))
    host = []
    for f in range(2):
        q, k, v = frames[(t + f) % pool]
        host.append(tuple([x[l].cpu().pin_memory() for l in range(L)] for x in (q, k, v)))
    host_out = torch.empty(L, H, n, d, dtype=torch.bfloat16).pin_memory()
    host_outs = [host_out[l] for l in range(L)]
    staging = torch.empty(xkv.xkv_stream_step_host_bytes(p, n), dtype=torch.uint8, device="cuda")

    def step_host(i: int) -> None:
        q, k, v = host[i % 2]
        xkv.xkv_stream_step_host(caches, q, k, v, host_outs, staging)

    for i in range(3):
        step_host(i)
    barrier()
    t0 = time.perf_counter()
    for i in range(Ke):
        step_host(i)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_s = max_over_ranks(e2e_s)
    frame_bytes = L * H * n * d * 2

    if rank == 0:
        peaks = _peaks()
        ms_step = ms_total / K
        attn_ms, attn_cnt = prof.get("attn", (0.0, 0))
        flops = 4.0 * n * w["budget"] * d * H                     # useful FLOPs of one attention launch
        attn_avg_s = (attn_ms / max(attn_cnt, 1)) * 1e-3
        achieved = flops / attn_avg_s / 1e12 if attn_avg_s > 0 else 0.0
        # the head means run on the library's side stream beside the attention: their event span in
        # the stream step is not a duration and is left out of the shares
        overlapped = ("kbar",)
        prof_total = sum(v[0] for k_, v in prof.items() if k_ not in overlapped)
        nbytes = maintenance_bytes(H, n, d, w["budget"], w["kv_bits"], w["key_mode"])

        def entry(ms: float, cnt: int, per: int, key: str | None, **extra) -> dict:
            e = dict(ms_per_step=ms / per, launches_per_step=cnt / per, avg_launch_us=ms / max(cnt, 1) * 1e3, **extra)
            if key in nbytes and ms > 0:
                sec = ms / cnt * 1e-3
                e.update(bytes_per_launch=nbytes[key], gb_per_s=nbytes[key] / sec / 1e9,
                         hbm_frac=nbytes[key] / sec / 1e9 / peaks["hbm_gbs"])
            return e

        kernels = {}
        for k_, v_ in prof.items():
            if not v_[1]:
                continue
            if k_ in overlapped:
                kernels[k_] = dict(launches_per_step=v_[1] / K, overlapped=True,
                                   note="event span beside the attention; see kernels_per_call.kbar for its duration")
            else:
                kernels[k_] = entry(v_[0], v_[1], K, k_, share=v_[0] / prof_total if prof_total else 0.0)
        per_call = {k_: entry(v_[0], v_[1], Kc, k_) for k_, v_ in calls.items() if v_[1] and k_ in ("append", "score_evict", "pack")}
        per_call["kbar"] = entry(kbar_alone[0], kbar_alone[1], 1, "kbar")
        line = dict(metric=METRIC, value=aggregate_frames_per_s(world, K, ms_total), unit=UNIT, n_gpus=world, steps=K, warmup=W,
                    ms_per_step=ms_step, higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f16",
                    data="synthetic",
                    config=dict(workload=w["name"], layers=L, heads=H, head_dim=d, tokens_per_frame=n,
                                budget=w["budget"], kv_bits=w["kv_bits"], keys="once" if w["key_mode"] else "regroup",
                                prefill_frames=fill, resident_frames=pool,
                                attention="unquantised_tail" if args.tail else "packed",
                                l2="inputs exceed L2 (about 1.2 GB touched per step)", replicas=world),
                    clocks=clocks.summary(),
                    e2e=dict(value=world * Ke / e2e_s, unit=UNIT, h2d_bytes_per_step=3 * frame_bytes,
                             d2h_bytes_per_step=frame_bytes, steps=Ke),
                    gpu_launches=int(launches),
                    roofline=dict(bound="tensor", kernel="attn_packed_causal", achieved=achieved,
                                  peak=peaks["tflops_sustained"], unit="TFLOP/s",
                                  frac=achieved / peaks["tflops_sustained"], peak_source=peaks["source"] + " (sustained)",
                                  frac_of_burst=achieved / peaks["tflops_burst"], flops_per_launch=flops,
                                  avg_launch_ms=attn_avg_s * 1e3,
                                  traffic=ATTN_DRAM_TRAFFIC_BYTES if w["name"] == WORKLOAD["name"] else None),
                    kernels=kernels, kernels_per_call=per_call)
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_uncompressed(args) -> None:
    """The growing-cache baseline of the ablation list: 16-bit storage and a budget that is never
    reached, i.e. no pruning and no quantisation, streamed from an empty cache.  The stream stops
    at --uncompressed-frames; the frame at which this layout would fill 90 % of the free device
    memory is computed, never provoked.  Prints one JSON line with the time of every 8th frame."""
    import torch
    import paper_2601_01204_b200.xkv as xkv
    from paper_2601_01204_b200 import synth
    if not torch.cuda.is_available():
        sys.exit("bench.py needs a CUDA device")
    w = dict(WORKLOAD)
    L, H, d, n, F = w["layers"], w["n_heads"], w["head_dim"], w["n_tokens"], args.uncompressed_frames
    p = xkv.Params(n_heads=H, head_dim=d, n_special=w["n_special"], pool_g=w["pool_g"], quant_group=w["quant_group"],
                   kv_bits=16, budget=F * n, max_frame_tokens=n)
    need = L * xkv.xkv_workspace_bytes(p)
    free, _ = torch.cuda.mem_get_info()
    per_frame = (L * xkv.xkv_workspace_bytes(xkv.Params(n_heads=H, head_dim=d, kv_bits=16, budget=2 * F * n,
                                                        max_frame_tokens=n)) - need) / F
    stop_frame = int((0.9 * free - (need - per_frame * F)) / per_frame)
    if need > 0.5 * free:
        sys.exit(f"refusing to hold {need / 1e9:.1f} GB of {free / 1e9:.1f} GB free: lower --uncompressed-frames")
    caches = [xkv.Cache(p) for _ in range(L)]
    pool = 4
    frames = []
    for f in range(pool):
        q = torch.empty(L, H, n, d, dtype=torch.bfloat16, device="cuda")
        k, v = torch.empty_like(q), torch.empty_like(q)
        for l in range(L):
            xkv.xkv_synth_fill(q[l], w["seed"] + l, l, f, synth.TENSOR_Q)
            xkv.xkv_synth_fill(k[l], w["seed"] + l, l, f, synth.TENSOR_K)
            xkv.xkv_synth_fill(v[l], w["seed"] + l, l, f, synth.TENSOR_V)
        frames.append(tuple([x[l] for l in range(L)] for x in (q, k, v)))
    out = torch.empty(L, H, n, d, dtype=torch.bfloat16, device="cuda")
    outs = [out[l] for l in range(L)]
    marks = []
    for t in range(F):
        q, k, v = frames[t % pool]
        if t % 8 == 7 or t == F - 1:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            xkv.xkv_stream_step(caches, q, k, v, outs)
            e1.record()
            marks.append((t + 1, e0, e1))
        else:
            xkv.xkv_stream_step(caches, q, k, v, outs)
    torch.cuda.synchronize()
    assert all(c.xkv_get_info().T == F * n and c.xkv_poll_status() == 0 for c in caches)
    print(json.dumps(dict(
        workload=f"uncompressed_bf16_growing_{L}L_{n}tok", frames=F, workspace_gb=need / 1e9,
        bytes_per_frame=per_frame, stop_frame_at_90pct_of_free_memory=stop_frame, free_gb=free / 1e9,
        ms_per_frame={str(t): round(a.elapsed_time(b), 3) for t, a, b in marks},
        note="this library keeps two buffer sets, so a frame costs twice the 135 MB of a single bf16 cache")),
        flush=True)


def maintenance_bytes(H: int, n: int, d: int, budget: int, bits: int, key_mode: int = 0) -> dict:
    """Bytes that one steady-state launch of each cache-maintenance launch has to move (4-bit cache):
    what it reads plus what it writes, every array once.  prunable = budget - n middle tokens are
    scored, k = budget - 2 n of them survive, n new tokens arrive.  Keys are the profile categories:
    the per-call launches (append, score_evict, pack), the head means (kbar) and the stream step's
    single launch (maint = append + pooled query + scores + selection + pack)."""
    if bits != 4:
        return {}
    row, code, par = d * 2, d // 2, 8                      # bf16 row, packed row, one (scale, zero) pair
    prunable, k = budget - n, max(0, budget - 2 * n)
    grp = lambda tokens: (tokens + 63) // 64 * d * par     # key parameters of the 64-token groups
    append = H * n * (2 * row) + H * n * (row + code + par)                 # K, V in; staged K, V codes + params out
    pool = H * n * row                                                     # Q in
    score = prunable * (4 * d + 4)                                         # stored head means in, scores out
    select = 2 * 4 * prunable + 4 * k                                      # scores read by both passes, kept out
    kbar = H * (prunable * code + grp(prunable)) + prunable * 4 * d        # codes + parameters in, head means out
    # keys regrouped (survivors' codes and parameters, new bf16 keys in; codes and parameters
    # out) and the survivors' value rows and parameters moved
    pack = H * (k * code + grp(k) + n * row + (k + n) * code + grp(k + n)) + 2 * H * k * (code + par)
    if key_mode == 1:
        # keys quantised once: the frame's key codes, group parameters and head means are written on
        # arrival; packing moves the survivors' code rows, value parameters and head-mean rows
        append = H * n * (2 * row) + H * n * (2 * code + par) + grp(n) * H * 2 + n * 4 * d
        pack = 2 * H * k * (2 * code + par) + 2 * k * (4 * d + 8)
        return {"append": append, "score_evict": pool + score + select, "pack": pack,
                "maint": append + pool + score + select + pack}
    return {"append": append, "score_evict": pool + kbar + score + select, "pack": pack, "kbar": kbar,
            "maint": append + pool + score + select + pack}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="xkv", choices=["xkv", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--budget", type=int, default=0, help="variant of the workload: token budget (ablation sweep)")
    ap.add_argument("--bits", type=int, default=0, choices=[0, 4, 8, 16],
                    help="variant: 4, 16 (prune only) or 8 (implies --keys once)")
    ap.add_argument("--tokens", type=int, default=0, help="variant: tokens per frame (1004 = long-stream shape)")
    ap.add_argument("--keys", default="regroup", choices=["regroup", "once"],
                    help="variant: keys re-quantised per 64-position run every step (default) or quantised once on arrival")
    ap.add_argument("--uncompressed-frames", type=int, default=0,
                    help="instead of the benchmark: stream this many frames through 16-bit caches that never prune")
    ap.add_argument("--tail", action="store_true",
                    help="variant: every frame attends to its own K, V unquantised (attn_packed_causal_tail)")
    ap.add_argument("--layers", type=int, default=0,
                    help="profiling aid: run a reduced stack of the same workload (default: all 24 layers)")
    args = ap.parse_args()
    if args.uncompressed_frames > 0:
        run_uncompressed(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_xkv(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the hybrid-KV decode path on B200.

Workload (N = 1): the LLaMA-3.1-8B-shaped single-layer decode at 32K context
(batch 1, 32 query / 8 KV heads, head_dim 128, bf16; per KV head 32 dims kept
per token, 96 dims held as M = 1024 Fourier coefficients; 4 sink + 1024 recent
tokens kept whole).  One STEP = one decode step of the whole hot path on a
resident cache through fa_decode_step: the new token is pushed (Eq.5: the
row that leaves the local window joins the middle and is added to every
coefficient row) and the query attends to the result (Eq.6).  The
cache of one layer (43 MB) would fit the 126 MB L2, so the steps rotate over
`--instances` independent caches (>= 8, > L2 in total).

Printed JSON (one line, rank 0): metric / value = microseconds per step,
device-timed with CUDA events around replays of a CUDA graph of exactly K steps
(median of `--replays`, min / max in `spread`); `per_config` = configurations 3
and 4 over 32 layers (fa_decode_step_layers, one cache per layer) and
configuration 2 as 32 fa_compress calls; `e2e_wall` = the host-buffer call made
eagerly, on the host clock;
`e2e` = the same through fa_decode_step_host with pinned HOST q / k_new /
v_new / out; `roofline` = fa_decode_attention alone (one fused kernel) against
the measured HBM peak on the bytes the hybrid cache holds; `cpu_baseline` = the
fp64 oracle on the host cores on a stated sample.  `--impl reference` times the
oracle instead.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "decode_attn_us_per_step_32k"
UNIT = "us/step"
SEED = 1000          # 1000 * config index


def _peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            p = json.load(f)
        return float(p["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while a region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def __enter__(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "50", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            self.thr = threading.Thread(target=self._read, daemon=True)
            self.thr.start()
        except Exception:
            self.proc = None
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def __exit__(self, *a):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self):
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0])); mx.append(float(r[1]))
                for n, v in zip(names, r[3:7]):
                    if v.lower().startswith("active"):
                        reasons.add(n)
            except Exception:
                continue
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def algorithmic_bytes(shape, n_mid: int, n_win: int) -> dict:
    """Bytes the hybrid cache holds and one decode / append call must move (per layer)."""
    eb = 2 if shape.dtype == "bf16" else 4
    d, M = shape.d, shape.M
    dck, dcv = d - shape.n_full_k, d - shape.n_full_v
    per_head = n_mid * (shape.n_full_k + shape.n_full_v) * eb + n_win * 2 * d * eb + M * (dck + dcv) * 4 + 2 * shape.G * d * eb
    append_head = 2 * M * (dck + dcv) * 4 + 4 * d * eb
    return {"decode": shape.B * shape.Hkv * per_head, "append": shape.B * shape.Hkv * append_head}


# ----------------------------------------------------------------- oracle arm
def oracle_sample_time(shape, seed: int, n_heads: int, L: int, repeats: int = 1):
    """Builds an oracle cache for the first n_heads KV heads and the first L tokens of the
    workload and times one step (append + decode) on it.  Returns (seconds per step, threads)."""
    import numpy as np
    from oracle import fa_oracle as fo
    from paper_2506_11886_b200 import synth
    sub = shape.with_(Hkv=n_heads, Hq=n_heads * shape.G, L=L)
    stream = synth.KVStream(sub, seed=seed)
    K, V = stream.tokens(0, L + repeats + 1)
    cfg = fo.OracleConfig(B=sub.B, Hq=sub.Hq, Hkv=sub.Hkv, d=sub.d, n_full_k=sub.n_full_k, n_full_v=sub.n_full_v,
                          k=sub.k, T=sub.T, L_init=sub.L_init, L_local=sub.L_local, cap_mid=sub.T, scale=sub.softmax_scale)
    cache = fo.OracleCache(cfg, stream.idx_full_k.numpy(), stream.idx_full_v.numpy())
    Kd, Vd = K.to(dtype=__import__("torch").float64).numpy(), V.to(dtype=__import__("torch").float64).numpy()
    cache.compress(Kd[:, :L], Vd[:, :L])
    times = []
    for r in range(repeats):
        q = synth.queries(sub, seed=seed, step=r).to(dtype=__import__("torch").float64).numpy()
        t0 = time.perf_counter()
        cache.append(Kd[:, L + r], Vd[:, L + r])
        out = cache.decode(q)
        times.append(time.perf_counter() - t0)
        assert np.isfinite(out).all()
    return times, fo.num_threads()


def run_reference(args):
    """The reference arm: the fp64 oracle, as it stands, on the host cores."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import fa_oracle as fo
    from paper_2506_11886_b200 import synth
    fo.build()
    shape = synth.CONFIGS[1]
    total = args.steps + args.warmup
    # bounded sample: one KV head, context truncated so that the whole run stays within ~2.5 minutes
    calib, threads = oracle_sample_time(shape, SEED, 1, 2048 + shape.L_init + shape.L_local, repeats=1)
    per_token = calib[0] / 2048.0
    budget = 150.0 / max(1, total)
    L_mid_full = shape.L - shape.L_init - shape.L_local
    n_mid = int(max(256, min(L_mid_full, budget / max(per_token, 1e-9))))
    L = n_mid + shape.L_init + shape.L_local
    times, threads = oracle_sample_time(shape, SEED, 1, L, repeats=total)
    timed = times[args.warmup:]
    scale = shape.Hkv * (L_mid_full / n_mid)
    sec = sum(timed) / len(timed)
    us = sec * scale * 1e6
    sample = f"1 of {shape.Hkv} KV heads, first {L} of {shape.L} tokens per step, time scaled x{scale:.1f}"
    line = {"metric": METRIC, "value": us, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": us / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "impl": "reference",
            "config": {"workload": shape.name, "global_batch": shape.B, "seq_len": shape.L, "sample": sample},
            "cpu_baseline": {"value": us, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": us, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# -------------------------------------------------------------------- our arm
PROFILE_FILES = {"decode_cfg1": "decode_cfg1_counters.md", "compress_cfg1": "compress_cfg1_counters.md"}


def profile_counter(file_key: str, section: str, label: str):
    """Reads one figure of a committed ncu summary under profiles/: the first line `* <label>: <number>`
    below the first heading that contains `section`.  None if the file, section or label is absent."""
    import re
    path = os.path.join(ROOT, "profiles", PROFILE_FILES[file_key])
    try:
        text = open(path).read()
    except OSError:
        return None
    m = re.search(r"^## .*" + re.escape(section) + r".*$", text, re.M)
    if not m:
        return None
    body = text[m.end():]
    nxt = re.search(r"^## ", body, re.M)
    if nxt:
        body = body[:nxt.start()]
    m = re.search(r"^\* " + re.escape(label) + r":\s*([-0-9.eE+]+)", body, re.M)
    return float(m.group(1)) if m else None


def make_layout(fa, shape):
    return fa.Layout(batch=shape.B, n_q_heads=shape.Hq, n_kv_heads=shape.Hkv, head_dim=shape.d, n_full_k=shape.n_full_k,
                     n_full_v=shape.n_full_v, n_coef=shape.M, period=shape.T, l_init=shape.L_init, l_local=shape.L_local,
                     max_mid=shape.T, mid_classes=shape.T // shape.k,
                     kv_dtype=fa.FA_BF16 if shape.dtype == "bf16" else fa.FA_F32, softmax_scale=shape.softmax_scale)


class Timer:
    """CUDA-graph timing on the launching stream: a warm-up graph, then `reps` timed replays of the
    graph of exactly n_steps steps, each between CUDA events; max over ranks per replay."""

    def __init__(self, torch, replicas, dev, reps):
        self.torch, self.replicas, self.dev, self.reps = torch, replicas, dev, reps

    def barrier(self):
        self.torch.cuda.synchronize()
        self.replicas.barrier()
        self.torch.cuda.synchronize()

    def graph(self, body, n_warm, n_steps, reps=None):
        torch = self.torch
        for s in range(2):
            body(s)                                   # eager: sets kernel attributes before any capture
        torch.cuda.synchronize()
        g_warm, g_time = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_warm):
            for s in range(n_warm):
                body(s)
        with torch.cuda.graph(g_time):
            for s in range(n_warm, n_warm + n_steps):
                body(s)
        g_warm.replay()
        ms = []
        for _ in range(reps or self.reps):
            self.barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g_time.replay()
            e1.record()
            self.barrier()
            ms.append(self.replicas.max_over_ranks(e0.elapsed_time(e1), device=self.dev))
        return ms


def spread(ms_list, n_steps):
    us = sorted(m * 1e3 / n_steps for m in ms_list)
    return {"median": statistics.median(us), "min": us[0], "max": us[-1], "replays": len(us)}


def bench_layers(torch, fa, synth, timer, dev, cfg_id, n_layers, tok_steps, warm, peak):
    """One configuration as the description states it: n_layers layers (one cache instance each), a
    token step = fa_decode_step_layers over all layers.  Returns the per_config entry."""
    shape = synth.CONFIGS[cfg_id]
    layout = make_layout(fa, shape)
    stream = synth.KVStream(shape, seed=SEED * cfg_id, device=str(dev))
    Kp, Vp = stream.tokens(0, shape.L, work_dtype=torch.float32)
    ws = fa.new_workspace(layout, device=dev)
    caches = []
    for i in range(n_layers):
        c = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v, device=dev)
        fa.fa_compress(layout, c, Kp, Vp, ws)
        caches.append(c)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    comp = []
    for _ in range(3):
        ev0.record(); fa.fa_compress(layout, caches[-1], Kp, Vp, ws); ev1.record(); torch.cuda.synchronize()
        comp.append(ev0.elapsed_time(ev1))
    del Kp, Vp
    n_mid0 = shape.L - shape.L_init - shape.L_local
    room = layout.max_mid - n_mid0
    reps = timer.reps
    per_replay = tok_steps
    assert (warm + 2 + per_replay * reps) <= room, "not enough room in the period for the timed appends"
    Kn, Vn = stream.tokens(shape.L, shape.L + 1, work_dtype=torch.float32)
    k_new, v_new = Kn[:, 0].contiguous(), Vn[:, 0].contiguous()
    qs = [synth.queries(shape, seed=SEED * cfg_id, step=i, layer=i, device=str(dev)) for i in range(n_layers)]
    outs = [torch.empty_like(q) for q in qs]
    args = fa.LayerStep([layout] * n_layers, caches, qs, [k_new] * n_layers, [v_new] * n_layers, outs)
    saved = [c.state.clone() for c in caches]

    def rewind():
        for c, st in zip(caches, saved):
            c.state.copy_(st)

    ms_tok = timer.graph(lambda s: fa.fa_decode_step_layers(args, ws), warm, tok_steps)
    rewind()

    def decode_all(s):
        for i in range(n_layers):
            fa.fa_decode_attention(layout, caches[i], qs[i], outs[i], ws)
    ms_dec = timer.graph(decode_all, warm, tok_steps)
    for c in caches:
        st = fa.fa_poll_status(c)
        assert st == fa.FA_OK, fa.status_string(st)
    assert all(torch.isfinite(o.float()).all() for o in outs)
    by = algorithmic_bytes(shape, n_mid0, shape.L_init + shape.L_local)
    tok = spread(ms_tok, tok_steps)
    dec = spread(ms_dec, tok_steps * n_layers)
    dec_gbs = by["decode"] / (dec["median"] * 1e-6) / 1e9
    comp_flop = 2.0 * shape.M * n_mid0 * ((shape.d - shape.n_full_k) + (shape.d - shape.n_full_v)) * shape.Hkv * shape.B
    out = {"workload": shape.name, "layers": n_layers, "us_per_token_step": tok["median"], "us_per_token_step_min": tok["min"],
           "us_per_token_step_max": tok["max"], "us_per_layer_step": tok["median"] / n_layers,
           "decode_us_per_layer": dec["median"], "algorithmic_bytes_per_layer": by["decode"],
           "hbm_bytes_per_token_step": by["decode"] * n_layers + by["append"] * n_layers,
           "decode_gbs": dec_gbs, "frac": dec_gbs / peak,
           "step_gbs": (by["decode"] + by["append"]) * n_layers / (tok["median"] * 1e-6) / 1e9,
           "tokens_per_s": shape.B * 1e6 / tok["median"],
           "launches_per_token_step": n_layers * fa.fa_launch_count(layout, 3),
           "compress_ms_per_layer": min(comp), "compress_tflops": comp_flop / (min(comp) * 1e-3) / 1e12}
    del caches, args
    torch.cuda.empty_cache()
    return out


def bench_compress_layers(torch, fa, synth, dev, n_layers, bf16_peak):
    """Configuration 2: prefill compression of n_layers layers, one cache per layer: as one fa_compress_layers call and
    as n_layers fa_compress calls."""
    shape = synth.CONFIGS[2]
    layout = make_layout(fa, shape)
    stream = synth.KVStream(shape, seed=SEED * 2, device=str(dev))
    Kp, Vp = stream.tokens(0, shape.L, work_dtype=torch.float32)
    ws = fa.new_workspace(layout, device=dev)
    caches = [fa.Cache(layout, stream.idx_full_k, stream.idx_full_v, device=dev) for _ in range(n_layers)]
    for c in caches[:2]:
        fa.fa_compress(layout, c, Kp, Vp, ws)
    layouts, Ks, Vs = [layout] * n_layers, [Kp] * n_layers, [Vp] * n_layers
    fa.fa_compress_layers(layouts, caches, Ks, Vs, ws)
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tot, single = [], []
    for _ in range(3):
        ev0.record()
        fa.fa_compress_layers(layouts, caches, Ks, Vs, ws)           # one call for the model's layers
        ev1.record()
        torch.cuda.synchronize()
        tot.append(ev0.elapsed_time(ev1))
        ev0.record()
        for c in caches:
            fa.fa_compress(layout, c, Kp, Vp, ws)                    # the same work as n_layers single calls
        ev1.record()
        torch.cuda.synchronize()
        single.append(ev0.elapsed_time(ev1))
    n_mid0 = shape.L - shape.L_init - shape.L_local
    flop = 2.0 * shape.M * n_mid0 * ((shape.d - shape.n_full_k) + (shape.d - shape.n_full_v)) * shape.Hkv * shape.B * n_layers
    tf = flop / (min(tot) * 1e-3) / 1e12
    tf1 = flop / (min(single) * 1e-3) / 1e12
    out = {"workload": shape.name, "layers": n_layers, "call": "fa_compress_layers (one call; the layers' kernels overlap)",
           "total_ms": min(tot), "ms_per_layer": min(tot) / n_layers,
           "useful_tflops": tf, "frac_of_bf16_tflops": tf / bf16_peak if bf16_peak else None,
           "single_calls_ms_per_layer": min(single) / n_layers, "single_calls_useful_tflops": tf1,
           "single_calls_frac_of_bf16_tflops": tf1 / bf16_peak if bf16_peak else None,
           "note": "same prefill tensor for every layer (3.1 GB of K/V per layer would not change the kernel's work)"}
    del caches, Kp, Vp
    torch.cuda.empty_cache()
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2506_11886_b200 import build, fa, replicas, synth

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    if not os.path.exists(fa.LIB_PATH):
        if rank == 0:
            build.build_library()
        if world > 1:
            dist.barrier()
    dev = torch.device("cuda", local)
    shape = synth.CONFIGS[args.config]
    K_steps, W = args.steps, max(args.warmup, 3)
    n_inst = max(args.instances, 2)
    layout = make_layout(fa, shape)
    stream = synth.KVStream(shape, seed=SEED, device=str(dev))
    Kp, Vp = stream.tokens(0, shape.L, work_dtype=torch.float32)
    ws = fa.new_workspace(layout, device=dev)
    caches = []
    for i in range(n_inst):
        c = fa.Cache(layout, stream.idx_full_k, stream.idx_full_v, device=dev)
        if i == 0:
            fa.fa_validate(layout, c)
        fa.fa_compress(layout, c, Kp, Vp, ws)
        caches.append(c)
    torch.cuda.synchronize()
    # compress timing (one layer of the 32-layer prefill-compression configuration has this exact shape)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    # (four calls back to back per sample, on four cache instances: a lone call would mostly time the launch of its first kernel)
    comp_ms = []
    for _ in range(3):
        ev0.record()
        for r in range(4):
            fa.fa_compress(layout, caches[-1 - (r % n_inst)], Kp, Vp, ws)
        ev1.record(); torch.cuda.synchronize()
        comp_ms.append(ev0.elapsed_time(ev1) / 4)
    n_mid0 = shape.L - shape.L_init - shape.L_local
    comp_flop = 2.0 * shape.M * n_mid0 * ((shape.d - shape.n_full_k) + (shape.d - shape.n_full_v)) * shape.Hkv * shape.B
    # the same compression by per-class transforms (FA_COMPRESS_FFT: fp32, order-fixed) and with ordered sums on the tensor path
    comp_fft_ms, comp_ord_ms = [], []
    for _ in range(3):
        for flags, acc in ((fa.FA_COMPRESS_FFT, comp_fft_ms), (fa.FA_COMPRESS_ORDERED, comp_ord_ms)):
            ev0.record()
            for r in range(4):
                fa.fa_compress(layout, caches[-1], Kp, Vp, ws, flags=flags)
            ev1.record(); torch.cuda.synchronize()
            acc.append(ev0.elapsed_time(ev1) / 4)
    fa.fa_compress(layout, caches[-1], Kp, Vp, ws)
    prefill_bytes = 2.0 * shape.B * shape.L * shape.Hkv * shape.d * (2 if shape.dtype == "bf16" else 4)
    # dimension selection (Sec. 3.4) on the same prefill: all-dims compression + reconstruction error + ranking
    sel_ms = []
    for _ in range(3):
        ev0.record(); sel = fa.fa_select_dims(layout, Kp, Vp); ev1.record(); torch.cuda.synchronize()
        sel_ms.append(ev0.elapsed_time(ev1))
    sel_ok = bool(torch.equal(sel[0].cpu(), stream.idx_full_k) and torch.equal(sel[2].cpu(), stream.idx_full_v))
    del Kp, Vp, sel
    # per-step inputs: visit r of an instance appends token L + r (a replay of a graph appends its tokens again)
    reps = max(1, args.replays)
    per_replay = (K_steps + n_inst - 1) // n_inst + 1
    room = layout.max_mid - n_mid0
    while reps > 1 and (W + 4 + per_replay * reps) > room:
        reps -= 1
    assert (W + 4 + per_replay * reps) <= room, "too many steps for the period of this configuration"
    visits = W + 4 + per_replay
    Kn, Vn = stream.tokens(shape.L, shape.L + visits, work_dtype=torch.float32)      # [B][visits][Hkv][d]
    Kn, Vn = Kn.transpose(0, 1).contiguous(), Vn.transpose(0, 1).contiguous()          # [visits][B][Hkv][d]
    n_q = W + K_steps
    qs = torch.stack([synth.queries(shape, seed=SEED, step=s, device=str(dev)) for s in range(min(n_q, 64))])
    outs = torch.empty((n_q,) + tuple(qs.shape[1:]), dtype=qs.dtype, device=dev)
    visit = [0] * n_inst
    saved_state = [c.state.clone() for c in caches]

    def rewind():
        """Token counters back to the prefill's (the appended rows stay; only the room in the period matters)."""
        torch.cuda.synchronize()
        for c, st in zip(caches, saved_state):
            c.state.copy_(st)
        for i in range(n_inst):
            visit[i] = 0

    def step(s, do_append=True, do_decode=True, one_instance=False):
        i = 0 if one_instance else s % n_inst
        if do_append and do_decode:
            fa.fa_decode_step(layout, caches[i], qs[s % qs.shape[0]], Kn[visit[i] % visits], Vn[visit[i] % visits], outs[s], ws)
            visit[i] += 1
        elif do_append:
            fa.fa_append(layout, caches[i], Kn[visit[i] % visits], Vn[visit[i] % visits])
            visit[i] += 1
        elif do_decode:
            fa.fa_decode_attention(layout, caches[i], qs[s % qs.shape[0]], outs[s], ws)

    timer = Timer(torch, replicas, dev, reps)
    with ClockSampler(local) as clk:
        ms_step = timer.graph(lambda s: step(s), W, K_steps)
        rewind()
        ms_decode = timer.graph(lambda s: step(s, do_append=False), W, K_steps)
        ms_append = timer.graph(lambda s: step(s, do_decode=False), W, K_steps)
        rewind()
        # the same decode call on ONE cache instance: whatever of its bytes the 126 MB L2 keeps is served from there
        ms_decode_warm = timer.graph(lambda s: step(s, do_append=False, one_instance=True), W, K_steps, reps=1)
        # end to end: host q / k_new / v_new in, host out, through the host-buffer C-ABI call
        staging = torch.empty(fa.fa_step_staging_bytes(layout), dtype=torch.uint8, device=dev)
        q_h = qs.cpu().pin_memory()
        out_h = torch.empty((n_q,) + tuple(qs.shape[1:]), dtype=qs.dtype).pin_memory()
        Kn_h, Vn_h = Kn.cpu().pin_memory(), Vn.cpu().pin_memory()

        def e2e_step(s):
            i = s % n_inst
            fa.fa_decode_step_host(layout, caches[i], q_h[s % q_h.shape[0]], Kn_h[visit[i] % visits], Vn_h[visit[i] % visits], out_h[s], staging, ws)
            visit[i] += 1
        ms_e2e = timer.graph(e2e_step, W, K_steps)
        rewind()
        # the same call made eagerly, timed on the host clock: launch cost included, the stream synchronised every step
        n_wall = min(K_steps, per_replay * n_inst - n_inst)
        for s in range(W):
            e2e_step(s)
        torch.cuda.synchronize()
        t_wall = time.perf_counter()
        for s in range(W, W + n_wall):
            e2e_step(s)
            torch.cuda.current_stream().synchronize()
        us_wall = (time.perf_counter() - t_wall) * 1e6 / max(1, n_wall)
        rewind()
        time.sleep(0.2)
    clocks = clk.summary()
    for c in caches:
        st = fa.fa_poll_status(c)
        assert st == fa.FA_OK, fa.status_string(st)
    assert torch.isfinite(outs[W:].float()).all() and torch.isfinite(out_h[W:W + n_wall].float()).all()

    sp_step, sp_dec, sp_app, sp_e2e = spread(ms_step, K_steps), spread(ms_decode, K_steps), spread(ms_append, K_steps), spread(ms_e2e, K_steps)
    us_step, us_decode, us_append, us_e2e = sp_step["median"], sp_dec["median"], sp_app["median"], sp_e2e["median"]
    by = algorithmic_bytes(shape, n_mid0, shape.L_init + shape.L_local)
    peak, peak_kind = _peaks()
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            bf16_peak = float(json.load(f)["bf16_tflops"])
    except Exception:
        bf16_peak = 1590.0
    dec_gbs = by["decode"] / (us_decode * 1e-6) / 1e9
    eb = 2 if shape.dtype == "bf16" else 4
    q_bytes = shape.B * shape.Hq * shape.d * eb
    kv_bytes = shape.B * shape.Hkv * shape.d * eb
    launches = K_steps * fa.fa_launch_count(layout, 3)
    n_dec = fa.fa_launch_count(layout, 2)
    # figures of the committed ncu captures (profiles/): DRAM bytes of one decode launch, tensor-pipe share of the compress kernel
    traffic = None
    if args.config == 1:
        rd, wr = profile_counter("decode_cfg1", "decode", "dram read"), profile_counter("decode_cfg1", "decode", "dram write")
        traffic = int(rd + wr) if rd is not None and wr is not None else None
    tensor_pct = profile_counter("compress_cfg1", "compress_tc", "tensor pipe % (active cycles)")
    line = {
        "metric": METRIC if args.config == 1 else f"decode_attn_us_per_step_cfg{args.config}", "value": us_step / world, "unit": UNIT,
        "n_gpus": world, "steps": K_steps, "warmup": W,
        "ms_per_step": us_step / 1e3, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
        "dtype": f"{shape.dtype} storage, f32 arithmetic", "data": "synthetic",
        "config": {"workload": shape.name, "global_batch": shape.B * world, "seq_len": shape.L,
                   "step": "fa_decode_step (append + decode), one layer", "parallelism": f"replicas x{world}",
                   "l2": f"inputs larger than L2: {n_inst} cache instances x {by['decode'] / 1e6:.1f} MB rotated",
                   "timing": f"CUDA events around each of {sp_step['replays']} replays of one CUDA graph of K steps; value = median"},
        "spread": {"step_us": sp_step, "decode_us": sp_dec, "append_us": sp_app, "e2e_us": sp_e2e},
        "breakdown": {"decode_us": us_decode, "decode_us_l2_warm": ms_decode_warm[0] * 1e3 / K_steps, "append_us": us_append, "tokens_per_s": 1e6 / us_step * shape.B * world,
                      "append_gbs": by["append"] / (us_append * 1e-6) / 1e9, "append_frac": by["append"] / (us_append * 1e-6) / 1e9 / peak,
                      "compress_ms_per_layer": min(comp_ms), "compress_tflops": comp_flop / (min(comp_ms) * 1e-3) / 1e12,
                      "compress_frac_of_bf16_tflops": comp_flop / (min(comp_ms) * 1e-3) / 1e12 / bf16_peak,
                      "compress_tensor_pipe_pct": tensor_pct,
                      "compress_path": "tcgen05.mma.cta_group::2 bf16 x bf16 -> f32 (TMEM), CTA pairs, basis tiles generated in registers",
                      "compress_fft_ms_per_layer": min(comp_fft_ms),
                      "compress_fft_frac_of_hbm": prefill_bytes / (min(comp_fft_ms) * 1e-3) / 1e9 / _peaks()[0],
                      "compress_ordered_ms_per_layer": min(comp_ord_ms),
                      "select_dims_ms": min(sel_ms), "select_dims_finds_generator_sets": sel_ok},
        "roofline": {"kernel": "fa_decode_attention (one fused cooperative kernel: u, token loop, merge)" if n_dec == 1 else
                     f"fa_decode_attention ({n_dec} kernels: u, token loop, merge)", "bound": "hbm",
                     "achieved": dec_gbs, "peak": peak, "unit": "GB/s", "frac": dec_gbs / peak, "peak_kind": peak_kind,
                     "algorithmic_bytes": by["decode"], "traffic": traffic,
                     "traffic_source": "profiles/" + PROFILE_FILES["decode_cfg1"] if traffic is not None else None,
                     "frac_of_8tbs_nominal": dec_gbs / 8000.0},
        "e2e": {"value": us_e2e / world, "unit": UNIT, "h2d_bytes_per_step": q_bytes + 2 * kv_bytes, "d2h_bytes_per_step": q_bytes},
        "e2e_wall": {"value": us_wall, "unit": UNIT, "steps": n_wall,
                     "what": "host clock around eager fa_decode_step_host + stream synchronise per step (launch cost included)"},
        "gpu_launches": launches, "clocks": clocks,
    }
    del caches, Kn, Vn, qs, outs
    torch.cuda.empty_cache()
    if rank == 0 and world == 1 and args.config == 1 and not args.no_per_config:
        tl = Timer(torch, replicas, dev, reps=5)
        per = {"cfg1": {"workload": shape.name, "layers": 1, "us_per_layer_step": us_step, "decode_us_per_layer": us_decode,
                        "algorithmic_bytes_per_layer": by["decode"], "decode_gbs": dec_gbs, "frac": dec_gbs / peak}}
        per["cfg2"] = bench_compress_layers(torch, fa, synth, dev, 32, bf16_peak)
        per["cfg3"] = bench_layers(torch, fa, synth, tl, dev, 3, 32, 8, 3, peak)
        per["cfg4"] = bench_layers(torch, fa, synth, tl, dev, 4, 32, 4, 3, peak)
        line["per_config"] = per
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import fa_oracle as fo
        fo.build()
        n_heads = min(4 if args.config == 1 else 1, shape.Hkv)
        times, threads = oracle_sample_time(shape, SEED, n_heads, shape.L, repeats=1)
        scale = shape.Hkv / n_heads
        line["cpu_baseline"] = {"value": times[0] * scale * 1e6, "unit": UNIT, "cores": threads, "kind": "oracle",
                                "sample": f"{n_heads} of {shape.Hkv} KV heads, full {shape.L}-token context, one step "
                                          f"({times[0]:.1f} s of CPU work), time scaled x{scale:.1f}"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=400)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--instances", type=int, default=8)
    ap.add_argument("--config", type=int, default=1, choices=[0, 1, 3, 4],
                    help="synthetic configuration (one layer of it); 1 is the headline workload, the others are for the per-configuration table")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-per-config", action="store_true", help="skip the 32-layer runs of configurations 2, 3 and 4")
    ap.add_argument("--replays", type=int, default=5, help="timed replays of each graph (the reported value is their median)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the MI hook on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mix|reference] [--no-extras]

A step is one mix_apply() over one synthetic decode batch (d = 4096, 256 one-token requests,
64 probes + 32 steering vectors, 25 % of rows unhooked).  A repeat is EXACTLY K such steps, replayed
as a CUDA graph on ROTATING hidden-state buffers (>= 512 MiB in total, four times the L2), so every
step finds its activations cold in L2; inputs are resident in HBM.  The repeat is timed again and
again (one CUDA event between repeats) until the region is at least 0.35 s long; `ms_per_step` is
the median repeat time / K, so the figure does not depend on K.  One JSON line goes to stdout
(rank 0); the roofline fractions of the other configurations are under `roofline.targets`.  With N > 1 every rank runs its own replica on its own
batch (rows are independent: no collective on the data path), time = max over ranks.
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
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import workloads as W  # noqa: E402

METRIC = "mi_hook_token_rows_per_s"
UNIT = "token-rows/s"
WORKLOAD = "decode: d=4096, T=256 (256 requests x 1 token), 64 probes + 32 steering vectors, 25% unhooked"
ROTATE_BYTES = 512 << 20
SAE_FLAGS = 2            # mix_config.flags of the SAE contexts of the extras / --workload runs: MIX_FLAG_RETILE_W_ENC
                         # (tile-contiguous copy of W_enc made at registration); --no-retile streams W_enc as given
# dram__bytes_read.sum + dram__bytes_write.sum of one probe_steer_team_kernel launch on the decode workload, from an
# ncu capture of this kernel (reads only: the steered rows are still dirty in L2 when the kernel ends).  Reported as
# `roofline.traffic`, labelled as not re-measured; the fraction itself uses the algorithmic bytes.
DECODE_DRAM_BYTES_PER_LAUNCH = 2410752


NOMINAL_HBM_GBS = 8000.0        # B200 HBM3e (DGX figure; HGX 7.7 TB/s): context beside the measured peak
NOMINAL_BF16_TFLOPS = 2250.0    # dense bf16


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return dict(hbm_gbs=float(j["hbm_gbs"]), bf16_tflops=float(j["bf16_tflops"]),
                    bf16_tflops_sustained=float(j.get("bf16_tflops_sustained", j["bf16_tflops"])), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


# ------------------------------------------------------------------------------ clocks
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, device_index: int):
        self.samples = []
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(device_index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "50"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL,
                text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) >= 7:
                self.samples.append((time.time(), parts))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()           # the exact child started above
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, t0, t1):
        inside = [p for (ts, p) in self.samples if t0 <= ts <= t1]
        pool = inside or [p for (_, p) in self.samples[-3:]]
        if not pool:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        def num(x):
            try:
                return float(x)
            except ValueError:
                return None
        sm = [num(p[0]) for p in pool if num(p[0]) is not None]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = sorted({n for p in pool for n, v in zip(names, p[3:7]) if v.lower().startswith("active")})
        pw = [num(p[2]) for p in pool if num(p[2]) is not None]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": num(pool[0][1]), "reasons": reasons,
                "power_w_max": max(pw) if pw else None, "samples": len(inside)}


# ------------------------------------------------------------------------------ helpers
def decode_bytes(w):
    """Algorithmic bytes of one decode-config launch: hidden rows read (probe + steer), steer rows
    written back, each distinct weight vector once, the slot map, the scores."""
    d = w.d_model
    rows_p = rows_s = 0
    used = set()
    for t in range(w.T_live):
        a = w.apps.get(int(w.token_slot[t]))
        if a is None:
            continue
        used.add(int(w.token_slot[t]))
        if a.kind == W.KIND_PROBE:
            rows_p += 1
        elif a.kind == W.KIND_STEER:
            rows_s += 1
    wbytes = sum((w.apps[s].n_classes if w.apps[s].kind == W.KIND_PROBE else 1) * d * 2 for s in used)
    return (rows_p + 2 * rows_s) * d * 2 + wbytes + 4 * w.T_max + 4 * rows_p, rows_p, rows_s


def capture_steps(m, hiddens, scores, idxs, stream):
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=stream):
        for i in idxs:
            m.apply(hiddens[i], scores[i], stream=stream)
    return g


def dist_max(x: float, world: int) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device="cuda" if torch.cuda.is_available() else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def dist_sum(x: float, world: int) -> float:
    if world == 1:
        return x
    import torch.distributed as dist
    t = torch.tensor([x], dtype=torch.float64, device="cuda" if torch.cuda.is_available() else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def barrier(world):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ------------------------------------------------------------------------------ oracle legs
def host_threads():
    """Threads the oracle may use: the process's affinity mask.  numpy's BLAS pool (the oracle's matrix
    products) is set to exactly that many, so the printed count is the one that ran."""
    n = len(os.sched_getaffinity(0)) if hasattr(os, "sched_getaffinity") else (os.cpu_count() or 1)
    used = n
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        threadpool_limits(limits=n)
        pools = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        used = max(pools) if pools else 1
    except Exception:
        pass
    return n, used


def oracle_leg(seconds_target=10.0, max_batches=10000):
    """Time the float64 oracle, as it stands, on whole decode batches for about `seconds_target` s."""
    from oracle import mi_hook as O
    wh = W.host(W.make_decode("cpu"))
    O.apply_hook(wh)                                   # warm-up (page in numpy / BLAS)
    n, t0 = 0, time.perf_counter()
    while True:
        O.apply_hook(wh)
        n += 1
        dt = time.perf_counter() - t0
        if dt >= seconds_target or n >= max_batches:
            break
    return dict(rows_per_s=n * wh.T_max / dt, batches=n, seconds=dt, rows=n * wh.T_max)


def oracle_sae_sample(w, n_sae_rows=4, n_other_rows=8, seed=0):
    """The oracle on a bounded sample of an SAE-carrying configuration (tensors on cuda are copied to the host
    first): `n_sae_rows` SAE rows of weight set 0 -- the oracle converts a whole encoder to float64 for however
    few rows it is given, so rows/s on a sample UNDERSTATES a full pass -- and a few rows of every other kind."""
    from oracle import mi_hook as O
    wh = W.host(w, only_groups={0})
    rng = np.random.default_rng(seed)
    sae_rows, other = [], []
    for t in range(w.T_live):
        a = w.apps.get(int(w.token_slot[t]))
        if a is not None and a.kind == W.KIND_SAE and a.group == 0:
            sae_rows.append(t)
        elif a is not None and a.kind != W.KIND_SAE:
            other.append(t)
    rows = list(rng.choice(sae_rows, size=min(n_sae_rows, len(sae_rows)), replace=False)) if sae_rows else []
    rows += list(rng.choice(other, size=min(n_other_rows, len(other)), replace=False)) if other else []
    t0 = time.perf_counter()
    O.apply_hook(wh, rows)
    dt = time.perf_counter() - t0
    n_sae_total = sum(1 for t in range(w.T_live) if (w.apps.get(int(w.token_slot[t])) is not None
                                                        and w.apps[int(w.token_slot[t])].kind == W.KIND_SAE))
    return {"rows": len(rows), "sae_rows": min(n_sae_rows, len(sae_rows)), "seconds": dt, "rows_per_s": len(rows) / dt,
            "extrapolated_full_batch_s": dt / max(len(rows), 1) * w.T_live,
            "extrapolation": "sample seconds per row x %d live rows (%d of them SAE rows); an upper estimate, the per-weight-set "
                             "float64 conversion of the encoder is spread over few rows in the sample" % (w.T_live, n_sae_total)}


def cpu_baseline_block(seconds_target):
    """cpu_baseline of the contract line: the oracle on whole decode batches (the line's own workload), plus its
    time on sampled rows of configs 2 and 3."""
    avail, used = host_threads()
    cb = oracle_leg(seconds_target)
    out = {"value": cb["rows_per_s"], "unit": UNIT, "cores": used, "cores_available": avail, "kind": "oracle",
           "threads": "numpy BLAS pool set to the affinity mask (%d); the row loop itself is one Python thread" % avail,
           "sample": "%d whole decode batches (%d rows) in %.1f s" % (cb["batches"], cb["rows"], cb["seconds"])}
    if torch.cuda.is_available():
        try:
            out["cfg2_sae_heavy_sample"] = oracle_sae_sample(W.make_sae_heavy("cuda"), n_sae_rows=4, n_other_rows=0)
            torch.cuda.empty_cache()
            out["cfg3_mixed_sample"] = oracle_sae_sample(W.make_mixed("cuda"), n_sae_rows=4, n_other_rows=8)
            torch.cuda.empty_cache()
        except Exception as e:
            out["sae_sample_error"] = repr(e)
    return out


def run_reference(args, rank, world):
    """--impl reference: the oracle on the host cores, same metric and config."""
    if rank != 0:
        return
    steps, warm = args.steps or 20, args.warmup if args.warmup is not None else 3
    from oracle import mi_hook as O
    avail, used = host_threads()
    wh = W.host(W.make_decode("cpu"))
    for _ in range(max(warm, 1)):
        O.apply_hook(wh)
    t0 = time.perf_counter()
    for _ in range(steps):
        O.apply_hook(wh)
    dt = time.perf_counter() - t0
    val = steps * wh.T_max / dt
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
            "warmup": warm, "ms_per_step": 1e3 * dt / steps, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic", "config": contract_config(),
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": used, "cores_available": avail, "kind": "oracle",
                             "sample": "%d whole decode batches (256 rows each); float64 CPU oracle, one whole batch per step" % steps},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------ extras
def time_stages(m, fn, reps=5):
    """Per-kernel milliseconds of one apply via the library's stage-event taps (best of reps)."""
    n = m.launches_per_apply()
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n + 1)]
    m.set_stage_events(evs)
    best = None
    for _ in range(reps):
        fn()
        torch.cuda.synchronize()
        ms = [evs[i].elapsed_time(evs[i + 1]) for i in range(n)]
        best = ms if best is None else [min(a, b) for a, b in zip(best, ms)]
    m.set_stage_events(None)
    return dict(zip(m.STAGES[:n], best))


def extras_sae(name, w, peaks, mixlib, extra_flags=0, w_enc_bytes_per_el=2.0, conditional=False):
    """SAE-carrying config: per-kernel times, encode flop rate and weight-stream bandwidth.
    conditional: the graph is captured with mix_apply_conditional (the SAE chain under a graph IF node)."""
    m = W.make_context(mixlib.Mix, w, flags=SAE_FLAGS | extra_flags)
    h = w.hidden.clone()
    scores = torch.zeros((w.T_max, max(w.C_max, 1)), dtype=torch.float32, device="cuda")
    def fn():
        h.copy_(w.hidden)
        m.apply(h, scores)
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    st = time_stages(m, fn)
    # whole call under graph replay
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            (m.apply_conditional if conditional else m.apply)(h, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    times = []
    for _ in range(11):
        h.copy_(w.hidden)
        e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    counts = {}
    for t in range(w.T_live):
        a = w.apps.get(int(w.token_slot[t]))
        if a is not None and a.kind == W.KIND_SAE:
            counts[a.group] = counts.get(a.group, 0) + 1
    flops = sum(2.0 * n * w.d_model * w.groups[g].d_sae for g, n in counts.items())
    wbytes = sum(w_enc_bytes_per_el * w.d_model * w.groups[g].d_sae for g in counts)
    enc_s = max(st["encode"], st.get("encode_pair", 0.0)) * 1e-3      # (of the two encode kernels one works, the other returns at once)
    status = m.get_status()
    m.destroy()
    layout = "8-bit E4M3 codes in blocks of 128, tile-ordered copy; 8-bit input" if extra_flags & 64 else (
        "8-bit E4M3 codes, tile-ordered copy") if extra_flags & 32 else (
        "tile-contiguous copy" if SAE_FLAGS & 2 else "as registered")
    return {"workload": name, "w_enc_layout": layout,
            "t_call_ms_graph": min(times), "t_call_ms_graph_median_of_11": float(np.median(times)),
            "stage_ms": st, "sae_rows_per_group": counts,
            "encode_tflops": flops / enc_s / 1e12, "encode_frac_bf16_peak": flops / enc_s / 1e12 / peaks["bf16_tflops"],
            "encode_weight_stream_gbs": wbytes / enc_s / 1e9,
            "encode_frac_hbm_peak": wbytes / enc_s / 1e9 / peaks["hbm_gbs"],
            "encode_frac_bf16_sustained": flops / enc_s / 1e12 / peaks["bf16_tflops_sustained"],
            "encode_frac_hbm_nominal": wbytes / enc_s / 1e9 / NOMINAL_HBM_GBS,
            "encode_frac_bf16_nominal": flops / enc_s / 1e12 / NOMINAL_BF16_TFLOPS,
            "token_rows_per_s": w.T_live / (min(times) * 1e-3), "status": status}


def run_replay(peaks, mixlib, n_replays, fp8a=False, fp8w=False):
    """Config 4: one captured graph at T_max = 2048, a fresh slot map and live count per replay.
    fp8w: 8-bit encoder, bf16 rows as two E4M3 operands (half the W_enc bytes, the bf16 tensor time).
    fp8a: 8-bit encoder and 8-bit encoder input (half the W_enc bytes; the tensor bound is taken at twice the
    measured bf16 rate, the nominal ratio of the two formats)."""
    w = W.make_replay("cuda", fp8=fp8a or fp8w, fp8_act=fp8a)
    m = W.make_context(mixlib.Mix, w, flags=SAE_FLAGS | (32 | 64 if fp8a else (32 if fp8w else 0)))
    T = w.T_max
    h = w.hidden.clone()
    scores = torch.zeros((T, 1), dtype=torch.float32, device="cuda")
    s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        m.apply(h, scores, stream=s)
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            m.apply(h, scores, stream=s)
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    slot_pin = torch.empty(T, dtype=torch.int32).pin_memory()
    rec, bad_status = [], 0
    for r in range(n_replays):
        token_slot, n_live = W.replay_map(w, r)
        slot_pin.copy_(torch.from_numpy(token_slot))
        m.set_slot_map(slot_pin, n_live)
        if r % 50 == 0:
            h.copy_(w.hidden)
        e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
        ms = e0.elapsed_time(e1)
        counts = {}
        for t in range(n_live):
            a = w.apps.get(int(token_slot[t]))
            if a is not None and a.kind == W.KIND_SAE:
                counts[a.group] = counts.get(a.group, 0) + 1
        wbytes = sum((1.0 if (fp8a or fp8w) else 2.0) * w.d_model * w.groups[gi].d_sae for gi in counts)
        flops = sum(2.0 * n * w.d_model * w.groups[gi].d_sae for gi, n in counts.items())
        bound_ms = max(wbytes / (peaks["hbm_gbs"] * 1e9),
                       flops / ((2.0 if fp8a else 1.0) * peaks["bf16_tflops"] * 1e12)) * 1e3
        rec.append((n_live, sum(counts.values()), len(counts), ms, bound_ms))
        if r % 10 == 9 or r == n_replays - 1:
            bad_status |= m.get_status()
    m.destroy()
    a = np.array(rec)
    live = a[a[:, 2] > 0]
    ratio = live[:, 4] / live[:, 3] if len(live) else np.array([0.0])
    return {"workload": "replay (config 4)" + (", 8-bit encoder and input" if fp8a else (", 8-bit encoder, bf16 rows" if fp8w else "")),
            "replays": n_replays, "status_or": bad_status,
            "n_live_covered": {"min": int(a[:, 0].min()), "max": int(a[:, 0].max()), "zero": bool((a[:, 0] == 0).any()),
                               "full": bool((a[:, 0] == T).any())},
            "below_0p75": [{"n_live": int(x[0]), "sae_rows": int(x[1]), "groups_live": int(x[2]), "ms": float(x[3]),
                            "bound_ms": float(x[4])} for x in live[np.argsort(ratio)[:8]] if x[4] / x[3] < 0.75],
            "t_call_ms": {"min": float(a[:, 3].min()), "p50": float(np.median(a[:, 3])), "p90": float(np.quantile(a[:, 3], 0.9)),
                          "max": float(a[:, 3].max())},
            "empty_replay_ms": float(a[a[:, 0] == 0][:, 3].min()) if (a[:, 0] == 0).any() else None,
            "bound_over_time": {"p10": float(np.quantile(ratio, 0.1)), "p50": float(np.median(ratio)),
                                "p90": float(np.quantile(ratio, 0.9))},
            "token_rows_per_s_mean": float(a[:, 0].sum() / (a[:, 3].sum() * 1e-3)),
            "worst": {"n_live": int(a[a[:, 3].argmax(), 0]), "sae_rows": int(a[a[:, 3].argmax(), 1]),
                      "groups_live": int(a[a[:, 3].argmax(), 2]), "ms": float(a[:, 3].max()),
                      "bound_ms": float(a[a[:, 3].argmax(), 4])}}


def extras_replace_decode(peaks, mixlib, small=False):
    """The decode as a gather: config 2 with the error term OFF, so every row is rebuilt from b_dec and the k = 64
    selected plus 16 edited W_dec rows (512 rows x 80 rows x 8 KiB = 320 MiB gathered).  Reported: the decode
    kernel's time between stage events and the gather's bytes over it.  small: a 4096-wide case for profiling."""
    w = W.make_sae_heavy("cuda", d_sae=16384, T=256, R=16, G=2) if small else W.make_sae_heavy("cuda", edit_hint=gpu_edit_hint)
    for a in w.apps.values():
        a.add_error = False
    m = W.make_context(mixlib.Mix, w, flags=SAE_FLAGS)
    h = w.hidden.clone()
    def fn():
        h.copy_(w.hidden)
        m.apply(h)
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    st = time_stages(m, fn)
    key = "tail" if "tail" in st else "decode"
    n_rows = int(sum(1 for t in range(w.T_live) if w.apps.get(int(w.token_slot[t])) is not None))
    k = max(sw.k for sw in w.groups.values())
    nbytes = float(n_rows) * (k + w.r_max) * w.d_model * 2 + float(n_rows) * w.d_model * 2
    status = m.get_status()
    m.destroy()
    return {"what": "config 2 with add_error = 0: %d rows x (k=%d + %d edited) W_dec rows of %d B gathered, row written" % (
                n_rows, k, w.r_max, w.d_model * 2),
            "stage": key, "decode_us": st[key] * 1e3, "bytes": nbytes, "gather_gbs": nbytes / st[key] / 1e6,
            "frac_hbm_peak": nbytes / st[key] / 1e6 / peaks["hbm_gbs"], "stage_ms": st, "status": status,
            "note": "the merge of the TopK candidates runs in the same kernel when the stage is `tail`"}


def extras_conditional(w, mixlib):
    """mix_apply vs mix_apply_conditional on one SAE-carrying context, with and without SAE rows live:
    graph replay, hidden state refreshed before every replay, best of 7."""
    sae_slots = [s for s, a in w.apps.items() if a.kind == W.KIND_SAE]
    full = np.asarray(w.token_slot, dtype=np.int32)
    no_sae = np.where(np.isin(full, sae_slots), -1, full).astype(np.int32)
    scores = torch.zeros((w.T_max, max(w.C_max, 1)), dtype=torch.float32, device="cuda")
    out = {"workload": w.name, "unit": "ms per replayed call",
           "rows_live": {"all_apps": int((full >= 0).sum()), "sae_rows_removed": int((no_sae >= 0).sum())}}
    for label, cond in (("mix_apply", False), ("mix_apply_conditional", True)):
        m = W.make_context(mixlib.Mix, w, flags=SAE_FLAGS)
        h = w.hidden.clone()
        s = torch.cuda.Stream(); s.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(s):
            m.apply(h, scores, stream=s)
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                (m.apply_conditional if cond else m.apply)(h, scores, stream=s)
        torch.cuda.current_stream().wait_stream(s)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        res = {}
        for name, slot_map in (("sae_rows_live", full), ("no_sae_row_live", no_sae)):
            m.set_slot_map(slot_map)
            best = 1e30
            for _ in range(7):
                h.copy_(w.hidden)
                e0.record(); g.replay(); e1.record(); torch.cuda.synchronize()
                best = min(best, e0.elapsed_time(e1))
            res[name] = best
        res["status"] = m.get_status()
        out[label] = res
        m.destroy()
    return out


def extras_multiclass(peaks, mixlib, small=False):
    """Multi-class probes alone on a large batch (every row hooked, requests of 256 consecutive rows dealt
    round-robin over the probes): the tensor-core probe kernel plus the pass of the streaming kernel that
    skips these rows.  Bytes counted: the hidden state once."""
    out = {}
    shapes = [(5120, 16384, 16, 8, 1.0)] if small else [(4096, 65536, 2, 4, 1.0), (4096, 65536, 16, 8, 1.0),
                                                        (4096, 65536, 32, 4, 1.0), (8192, 32768, 8, 4, 1.0),
                                                        (5120, 16384, 16, 8, 1.0), (4096, 65536, 16, 8, 0.25)]
    for d, T, C, n_probe, density in shapes:
        g = torch.Generator(device="cuda"); g.manual_seed(1)
        hidden = torch.randn((T, d), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        m = mixlib.Mix(d_model=d, T_max=T, n_slots_max=n_probe, C_max=C)
        keep = []
        for s_ in range(n_probe):
            Wp = (torch.randn((C, d), generator=g, device="cuda") * d ** -0.5).to(torch.bfloat16); keep.append(Wp)
            m.register_probe(s_, Wp, None, mixlib.MIX_ACT_SOFTMAX)
        req = np.arange(T) // 256                                           # requests of 256 rows
        slot_map = (req % n_probe).astype(np.int32)
        if density < 1.0:                                                    # every (1/density)-th request is hooked
            slot_map = np.where(req % int(round(1 / density)) == 0, (req // int(round(1 / density))) % n_probe, -1).astype(np.int32)
        m.set_slot_map(torch.from_numpy(slot_map).cuda())
        scores = torch.zeros((T, C), dtype=torch.float32, device="cuda")
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best = 1e9
        for _ in range(6):
            e0.record(); m.apply(hidden, scores); e1.record(); torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        nbytes = int((slot_map >= 0).sum()) * d * 2                        # hooked rows only
        # the same call replayed from a CUDA graph (the serving way: no host time between the launches)
        gs = torch.cuda.Stream(); gs.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(gs):
            m.apply(hidden, scores, stream=gs)
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=gs):
                m.apply(hidden, scores, stream=gs)
        torch.cuda.current_stream().wait_stream(gs)
        torch.cuda.synchronize()
        for _ in range(3):                                                  # untimed: the first replays of a new graph run slow
            graph.replay()
        torch.cuda.synchronize()
        reps = []
        for _ in range(11):
            e0.record(); graph.replay(); e1.record(); torch.cuda.synchronize()
            reps.append(e0.elapsed_time(e1))
        graph_ms = float(np.median(reps))
        del graph
        st = time_stages(m, lambda: m.apply(hidden, scores))
        tc_ms = st["probe_tc"]
        out["d=%d T=%d C=%d probes=%d hooked=%d%%" % (d, T, C, n_probe, round(100 * density))] = {
            "ms": best, "gbs": nbytes / best / 1e6, "frac_hbm_peak": nbytes / best / 1e6 / peaks["hbm_gbs"],
            "graph_replay": {"ms_median_of_11": graph_ms, "frac_hbm_peak": nbytes / graph_ms / 1e6 / peaks["hbm_gbs"]},
            "frac_hbm_nominal": nbytes / best / 1e6 / NOMINAL_HBM_GBS, "stage_ms": st,
            "probe_tc_kernel_alone": {"gbs": nbytes / tc_ms / 1e6, "frac_hbm_peak": nbytes / tc_ms / 1e6 / peaks["hbm_gbs"]},
            "status": m.get_status()}
        m.destroy()
        del hidden
        torch.cuda.empty_cache()
    return out


def run_workload(args):
    """--workload X: one of the other configurations alone (not the contract line)."""
    import paper_2607_22595_b200 as mixlib
    from paper_2607_22595_b200 import _build
    _build.build()
    torch.cuda.set_device(0)
    peaks = measured_peaks()
    name = args.workload
    if name == "sweep":
        out = extras_sweep(peaks, mixlib)
    elif name == "sweep_small":       # profiling case for the streaming probe / steering kernel
        out = extras_sweep(peaks, mixlib, small=True)
    elif name == "sae_heavy":
        out = extras_sae("sae_heavy (config 2)", W.make_sae_heavy("cuda"), peaks, mixlib)
    elif name == "sae_heavy_fp8":   # config 2 with the encoder as 8-bit codes (MIX_FLAG_FP8_W_ENC)
        out = extras_sae("sae_heavy (config 2), 8-bit encoder", W.make_sae_heavy("cuda", fp8=True), peaks, mixlib,
                         extra_flags=32, w_enc_bytes_per_el=1.0)
    elif name == "mixed_fp8":
        out = extras_sae("mixed (config 3), 8-bit encoder", W.make_mixed("cuda", fp8=True), peaks, mixlib,
                         extra_flags=32, w_enc_bytes_per_el=1.0)
    elif name == "sae_small_fp8":   # profiling case for the 8-bit encoder
        out = extras_sae("sae_small, 8-bit encoder (d=4096, d_sae=16384, 2 sets, T=256)",
                         W.make_sae_heavy("cuda", d_sae=16384, T=256, R=16, G=2, fp8=True), peaks, mixlib,
                         extra_flags=32, w_enc_bytes_per_el=1.0)
    elif name == "sae_heavy_fp8a":  # config 2, 8-bit encoder AND 8-bit encoder input (E4M3 x E4M3 contraction)
        out = extras_sae("sae_heavy (config 2), 8-bit encoder and input", W.make_sae_heavy("cuda", fp8=True, fp8_act=True),
                         peaks, mixlib, extra_flags=32 | 64, w_enc_bytes_per_el=1.0)
    elif name == "mixed_fp8a":
        out = extras_sae("mixed (config 3), 8-bit encoder and input", W.make_mixed("cuda", fp8=True, fp8_act=True),
                         peaks, mixlib, extra_flags=32 | 64, w_enc_bytes_per_el=1.0)
    elif name == "sae_small_fp8a":  # profiling case for the 8-bit contraction
        out = extras_sae("sae_small, 8-bit encoder and input (d=4096, d_sae=16384, 2 sets, T=256)",
                         W.make_sae_heavy("cuda", d_sae=16384, T=256, R=16, G=2, fp8=True, fp8_act=True), peaks, mixlib,
                         extra_flags=32 | 64, w_enc_bytes_per_el=1.0)
    elif name == "mixed_small_fp8a":
        out = extras_sae("mixed_small, 8-bit encoder and input (d=5120, d_sae=8192, T=4096)",
                         W.make_mixed("cuda", T=4096, d_sae=8192, R=32, fp8=True, fp8_act=True), peaks, mixlib,
                         extra_flags=32 | 64, w_enc_bytes_per_el=1.0)
    elif name == "sae_small":     # profiling case: weights (256 MiB) exceed L2, < 1 GiB on the device
        out = extras_sae("sae_small (d=4096, d_sae=16384, 2 sets, T=256)",
                         W.make_sae_heavy("cuda", d_sae=16384, T=256, R=16, G=2), peaks, mixlib)
    elif name == "mixed":
        out = extras_sae("mixed (config 3)", W.make_mixed("cuda"), peaks, mixlib)
    elif name == "mixed_edit_only":   # config 3 with MIX_FLAG_SAE_EDIT_ONLY (an algorithmic shortcut, never a tensor-pipe figure)
        out = extras_sae("mixed (config 3), edit-only shortcut", W.make_mixed("cuda"), peaks, mixlib, extra_flags=8)
    elif name == "mixed_small":   # profiling case for the tensor-bound regime
        out = extras_sae("mixed_small (d=5120, d_sae=8192, T=4096)",
                         W.make_mixed("cuda", T=4096, d_sae=8192, R=32), peaks, mixlib)
    elif name == "conditional":   # the SAE chain as a graph IF node (config 3's context)
        out = extras_conditional(W.make_mixed("cuda"), mixlib)
    elif name == "conditional_small":
        out = extras_conditional(W.make_mixed("cuda", T=4096, d_sae=8192, R=32), mixlib)
    elif name == "multiclass":
        out = extras_multiclass(peaks, mixlib)
    elif name == "multiclass_small":   # profiling case: 168 MB of hidden state
        out = extras_multiclass(peaks, mixlib, small=True)
    elif name == "replace_decode":
        out = extras_replace_decode(peaks, mixlib)
    elif name == "replace_decode_small":   # profiling case
        out = extras_replace_decode(peaks, mixlib, small=True)
    elif name == "replay":
        out = run_replay(peaks, mixlib, args.steps or 200)
    elif name == "replay_fp8a":
        out = run_replay(peaks, mixlib, args.steps or 200, fp8a=True)
    elif name == "replay_fp8":
        out = run_replay(peaks, mixlib, args.steps or 200, fp8w=True)
    else:
        raise SystemExit("unknown workload %r" % name)
    print(json.dumps(out), flush=True)


def extras_decode_variants(w, hiddens, scores, mixlib):
    """The decode config with its apps gated / turned into projections: L2-cold µs per step."""
    T = w.T_max
    R = len(hiddens)
    out = {}
    g = torch.Generator(device="cuda"); g.manual_seed(7)
    gate_scores = torch.randn((T, 1), generator=g, device="cuda")          # about half of the gates open

    def measure(m):
        stream = torch.cuda.Stream(); stream.wait_stream(torch.cuda.current_stream())
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        with torch.cuda.stream(stream):
            m.apply(hiddens[0], scores[0], stream=stream)
            gr = capture_steps(m, hiddens, scores, range(R), stream)
            gr.replay()
            e0.record(stream)
            for _ in range(8):
                gr.replay()
            e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) * 1e3 / (8 * R)

    m = W.make_context(mixlib.Mix, w)
    for s in w.apps:
        m.set_gate(s, gate_scores, 0, mixlib.MIX_GATE_GE, 0.0)
    out["all_apps_gated_us_per_step"] = measure(m)
    m.destroy()
    m = W.make_context(mixlib.Mix, w)
    for s, a in w.apps.items():
        if a.kind == W.KIND_STEER:
            m.register_project(s, a.v, 1.0)
    out["steer_as_projection_us_per_step"] = measure(m)
    m.destroy()
    # several apps on one row: every hooked row gets a probe AND a steering vector, (a) as a slot
    # chain in one call (the row is read once), (b) as two contexts applied one after the other
    probes = [s for s, a in w.apps.items() if a.kind == W.KIND_PROBE]
    steers = [s for s, a in w.apps.items() if a.kind == W.KIND_STEER]
    slot = np.asarray(w.token_slot).copy()
    hooked = slot >= 0
    slot[hooked] = np.asarray(probes, dtype=np.int32)[np.arange(int(hooked.sum())) % len(probes)]
    wc = W.Workload("decode, probe -> steer on every hooked row", w.d_model, T, T, w.hidden, slot, w.apps, {},
                    n_slots_max=w.n_slots_max, C_max=1, chains={p: steers[i % len(steers)] for i, p in enumerate(probes)})
    m = W.make_context(mixlib.Mix, wc, flags=mixlib.MIX_FLAG_SLOT_CHAINS)
    out["probe_then_steer_chained_one_call_us_per_step"] = measure(m)
    m.destroy()
    link = {p: steers[i % len(steers)] for i, p in enumerate(probes)}
    slot_b = np.where(hooked, np.asarray([link.get(int(x), -1) for x in slot], dtype=np.int32), -1).astype(np.int32)
    ma = W.make_context(mixlib.Mix, W.Workload("a", w.d_model, T, T, w.hidden, slot, w.apps, {}, n_slots_max=w.n_slots_max))
    mb = W.make_context(mixlib.Mix, W.Workload("b", w.d_model, T, T, w.hidden, slot_b, w.apps, {}, n_slots_max=w.n_slots_max))

    class Two:
        def apply(self, h, sc, stream=None):
            ma.apply(h, sc, stream=stream)
            mb.apply(h, sc, stream=stream)
    out["probe_then_steer_two_calls_us_per_step"] = measure(Two())
    ma.destroy(); mb.destroy()
    # 32 hooked layers: 32 contexts (one per layer, same apps) applied one after the other to the decode step's
    # hidden state, all in the captured graph; per decode step, i.e. per 32 hook calls
    layers = [W.make_context(mixlib.Mix, w) for _ in range(32)]

    class Stack:
        def apply(self, h, sc, stream=None):
            for mm in layers:
                mm.apply(h, sc, stream=stream)
    out["32_hooked_layers_us_per_decode_step"] = measure(Stack())
    # changing one per-request parameter between replays, host cost per replay of a one-kernel graph: a 4-byte
    # write into a device table (what this library does) vs a kernel-node parameter update (the paper's way)
    tab, node = layers[0].bench_param_update(iters=3000)
    out["param_change_plus_graph_launch_us"] = {"device_table_write": tab, "kernel_node_param_update": node}
    for mm in layers:
        mm.destroy()
    return out


def extras_sweep(peaks, mixlib, small=False):
    """Bandwidth kernels alone at a size that cannot hide in L2: d = 8192, T = 65536, every row hooked.
    small: T = 16384 (256 MiB of hidden state) and no encode -- the profiling case."""
    d, T = 8192, (16384 if small else 65536)
    g = torch.Generator(device="cuda"); g.manual_seed(1)
    hidden = torch.randn((T, d), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    v = torch.randn((d,), generator=g, device="cuda").to(torch.bfloat16)
    Wp = (torch.randn((1, d), generator=g, device="cuda") * d ** -0.5).to(torch.bfloat16)
    m = mixlib.Mix(d_model=d, T_max=T, n_slots_max=2)
    m.register_steer(0, v, 2.0)
    m.register_probe(1, Wp, None, mixlib.MIX_ACT_SIGMOID)
    scores = torch.zeros((T, 1), dtype=torch.float32, device="cuda")
    out = {}
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for name, slot, nbytes in (("steer", 0, 2.0 * T * d * 2), ("probe", 1, 1.0 * T * d * 2)):
        m.set_slot_map(torch.full((T,), slot, dtype=torch.int32, device="cuda"))
        best = 1e9
        for _ in range(6):
            e0.record(); m.apply(hidden, scores); e1.record(); torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        out[name] = {"ms": best, "gbs": nbytes / best / 1e6, "frac_hbm_peak": nbytes / best / 1e6 / peaks["hbm_gbs"],
                     "frac_hbm_nominal": nbytes / best / 1e6 / NOMINAL_HBM_GBS}
    m.destroy()
    del hidden
    torch.cuda.empty_cache()
    if small:
        return out
    # the encode alone in the tensor-bound regime: one TopK weight set, every row an SAE row
    d, T, S = 4096, 4096, 65536
    sae = W.make_sae_weights(g, "cuda", d, S, W.SAE_TOPK, k=64)
    hidden = torch.randn((T, d), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    app = W.SaeApp(0, np.zeros(0, np.int32), np.zeros(0, np.float32), np.zeros(0, np.uint8), True)
    ws = W.Workload("encode alone", d, T, T, hidden, np.zeros(T, dtype=np.int32), {0: app}, {0: sae}, n_slots_max=1,
                    n_groups_max=1, C_max=1, k_max=64, r_max=1, d_sae_max=S)
    m = W.make_context(mixlib.Mix, ws, flags=SAE_FLAGS)
    h = hidden.clone()
    for _ in range(2):
        m.apply(h)
    torch.cuda.synchronize()
    st = time_stages(m, lambda: m.apply(h))
    flops = 2.0 * T * d * S
    enc_s = max(st["encode"], st.get("encode_pair", 0.0)) * 1e-3      # (of the two encode kernels one works, the other returns at once)
    out["encode"] = {"shape": "M=4096, d=4096, S=65536, one TopK weight set", "ms": enc_s * 1e3, "tflops": flops / enc_s / 1e12,
                     "frac_bf16_peak": flops / enc_s / 1e12 / peaks["bf16_tflops"],
                     "frac_bf16_sustained": flops / enc_s / 1e12 / peaks["bf16_tflops_sustained"],
                     "frac_bf16_nominal": flops / enc_s / 1e12 / NOMINAL_BF16_TFLOPS, "status": m.get_status()}
    m.destroy()
    return out


# ------------------------------------------------------------------------------ main arm
MIN_REGION_S = 0.35        # the timed region is repeated until it is at least this long


def plan_pass(m, hiddens, scores, K, stream):
    """Graphs whose replay, one after the other, is a whole number of repeats of EXACTLY K consecutive steps on
    rotating hidden buffers: returns (graphs, repeats per pass).  K <= number of buffers R (a multiple of K): one
    graph that walks all R buffers = R / K repeats back to back -- a K-step graph launched on its own would add
    the launch latency of a whole graph to every K steps, which belongs to the engine's graph, not to the hook
    kernel inside it; this way the per-step figure is the same for every K.  Larger K: the all-buffers graph
    replayed K // R times plus a remainder graph = one repeat.  Either way a buffer comes round again only after
    all the others (>= 4x L2) have been touched."""
    R = len(hiddens)
    if K <= R:
        return [capture_steps(m, hiddens, scores, range(R), stream)], R // K
    graphs = [capture_steps(m, hiddens, scores, range(R), stream)] * (K // R)
    if K % R:
        graphs.append(capture_steps(m, hiddens, scores, range(K % R), stream))
    return graphs, 1


def time_passes(graphs, n_pass, stream):
    """Replays the pass n_pass times back to back on `stream`, one CUDA event between consecutive passes.
    Returns the per-pass milliseconds."""
    evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_pass + 1)]
    with torch.cuda.stream(stream):
        evs[0].record(stream)
        for r in range(n_pass):
            for g in graphs:
                g.replay()
            evs[r + 1].record(stream)
    torch.cuda.synchronize()
    return [evs[r].elapsed_time(evs[r + 1]) for r in range(n_pass)]


def passes_for(graphs, stream, min_region_s=MIN_REGION_S):
    """Untimed: the pass twice (uploads the graphs), then a short estimate of its time."""
    time_passes(graphs, 2, stream)
    est_ms = float(np.median(time_passes(graphs, 3, stream)))
    return int(min(max(np.ceil(min_region_s * 1e3 / max(est_ms, 1e-3)), 5), 20000))


def contract_config():
    """The same in both arms (the driver compares them)."""
    return {"workload": WORKLOAD,
            "l2": "inputs larger than L2: the hidden states of successive steps rotate over >= 512 MiB of buffers "
                  "(4x L2), so every step finds its rows cold; the 0.75 MiB of weights stay warm, as in serving"}


def run_mix(args, rank, world, local_rank):
    import paper_2607_22595_b200 as mixlib
    from paper_2607_22595_b200 import _build
    _build.build()
    torch.cuda.set_device(local_rank)
    peaks = measured_peaks()
    w = W.make_decode("cuda", seed=W.BASE_SEED + 1000 + rank)
    m = W.make_context(mixlib.Mix, w)
    T, d = w.T_max, w.d_model
    K = args.steps or 256                      # steps per repeat
    Wm = max(args.warmup if args.warmup is not None else 5, 3)
    R = max(2, -(-ROTATE_BYTES // (T * d * 2)))
    if K < R:
        R = -(-R // K) * K                     # a whole number of K-step graphs
    hiddens = [w.hidden.clone() for _ in range(R)]
    scores = [torch.zeros((T, 1), dtype=torch.float32, device="cuda") for _ in range(R)]

    stream = torch.cuda.Stream()
    stream.wait_stream(torch.cuda.current_stream())
    # `value` is the step as it costs behind ANY predecessor kernel: the hook kernel launched the ordinary way.
    # (With programmatic dependent launch, hook calls placed back to back hide each other's table look-ups; that
    # figure is measured afterwards and reported beside it.)
    pdl_default = mixlib.set_pdl_mask(-1)
    mixlib.set_pdl_mask(pdl_default & ~8)
    with torch.cuda.stream(stream):
        for i in range(Wm):
            m.apply(hiddens[i % R], scores[i % R], stream=stream)   # W untimed warm-up steps, eager
        graphs, reps_per_pass = plan_pass(m, hiddens, scores, K, stream)
    torch.cuda.synchronize()
    n_pass = passes_for(graphs, stream)
    n_rep = n_pass * reps_per_pass

    sampler = ClockSampler(local_rank)
    time.sleep(0.3)
    barrier(world); torch.cuda.synchronize()
    t0 = time.time()
    per_rep = [x / reps_per_pass for x in time_passes(graphs, n_pass, stream)]     # ms per K steps
    barrier(world)
    t1 = time.time()
    ms_rep = dist_max(float(np.median(per_rep)), world)          # K steps, median over repeats, slowest rank
    ms_per_step = ms_rep / K
    rows_per_rep = dist_sum(float(K) * w.T_live, world)
    clocks = sampler.summary(t0, t1)
    region_s = float(np.sum(per_rep)) * reps_per_pass * 1e-3
    spread = {"p10": float(np.quantile(per_rep, 0.1)) / K * 1e3, "p50": float(np.median(per_rep)) / K * 1e3,
              "p90": float(np.quantile(per_rep, 0.9)) / K * 1e3, "mean": float(np.mean(per_rep)) / K * 1e3}

    def us_per_step(gs, steps_per_pass):
        n = passes_for(gs, stream, MIN_REGION_S / 3)
        return float(np.median(time_passes(gs, n, stream))) / steps_per_pass * 1e3

    # side figures, same protocol: (a) programmatic dependent launch of the hook kernel, calls back to back
    mixlib.set_pdl_mask(pdl_default)
    with torch.cuda.stream(stream):
        graphs_pdl, _ = plan_pass(m, hiddens, scores, K, stream)
    torch.cuda.synchronize()
    pdl_us = us_per_step(graphs_pdl, K * reps_per_pass)
    del graphs_pdl
    mixlib.set_pdl_mask(pdl_default & ~8)
    # (b) warm L2: every step on the same buffer
    Kw = 256
    with torch.cuda.stream(stream):
        graphs_warm = [capture_steps(m, hiddens, scores, [0] * Kw, stream)]
    torch.cuda.synchronize()
    warm_us = us_per_step(graphs_warm, Kw)
    # (c) launch floor: the same graphs with zero live rows (every CTA exits after one 4-byte load)
    m.set_slot_map(torch.from_numpy(w.token_slot.copy()).cuda(), 0)
    floor_us = us_per_step(graphs, K * reps_per_pass)
    m.set_slot_map(torch.from_numpy(w.token_slot.copy()).cuda(), w.T_live)
    torch.cuda.synchronize()
    del graphs_warm
    mixlib.set_pdl_mask(pdl_default)

    # end to end through the public API with host buffers: every step copies its hidden states
    # and slot map from pinned host memory, applies the hook, and copies hidden + scores back.
    # Steps are independent batches, so they are pipelined over a few contexts (one stream and
    # one device buffer each): the H2D of one step overlaps the D2H of another, as a serving
    # engine with several batches in flight would do.
    n_pipe = 3
    pipes = []
    for i in range(n_pipe):
        mi = m if i == 0 else W.make_context(mixlib.Mix, w)
        h_in = torch.empty((T, d), dtype=torch.bfloat16).pin_memory(); h_in.copy_(w.hidden.cpu())
        pipes.append(dict(m=mi, st=torch.cuda.Stream(), h_in=h_in,
                          h_out=torch.empty((T, d), dtype=torch.bfloat16).pin_memory(),
                          s_out=torch.empty((T, 1), dtype=torch.float32).pin_memory(),
                          slot=torch.from_numpy(w.token_slot.copy()).pin_memory(), hd=hiddens[i], sd=scores[i]))
    def e2e_step(i):
        p = pipes[i % n_pipe]
        torch.cuda.set_stream(p["st"])          # cheaper per step than the stream context manager
        p["hd"].copy_(p["h_in"], non_blocking=True)
        p["m"].set_slot_map(p["slot"], w.T_live, stream=p["st"])
        p["m"].apply(p["hd"], p["sd"], stream=p["st"])
        p["h_out"].copy_(p["hd"], non_blocking=True)
        p["s_out"].copy_(p["sd"], non_blocking=True)
    torch.cuda.synchronize()
    for i in range(2 * n_pipe):
        e2e_step(i)
    # host <-> device copies share the PCIe link and the host's memory system with other tenants of the box:
    # three rounds of max(K, 200) steps each, the fastest is reported
    n_round, K_e2e = 3, max(K, 200)
    e2e_s = None
    for _ in range(n_round):
        torch.cuda.synchronize(); barrier(world)
        te = time.perf_counter()
        for i in range(K_e2e):
            e2e_step(i)
        torch.cuda.synchronize()
        dt = dist_max(time.perf_counter() - te, world)
        e2e_s = dt if e2e_s is None else min(e2e_s, dt)
    torch.cuda.set_stream(torch.cuda.default_stream())
    sampler.stop()
    e2e_rows = dist_sum(float(K_e2e) * w.T_live, world)
    status = m.get_status()

    if rank != 0:
        return
    nbytes, rows_p, rows_s = decode_bytes(w)
    achieved = nbytes / (ms_per_step * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": rows_per_rep / (ms_rep * 1e-3), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic", "config": contract_config(),
        "clocks": clocks,
        "e2e": {"value": e2e_rows / e2e_s, "unit": UNIT, "h2d_bytes_per_step": T * d * 2 + 4 * T,
                "d2h_bytes_per_step": T * d * 2 + 4 * T, "steps": K_e2e, "rounds": "fastest of %d" % n_round,
                "pipeline_depth": n_pipe},
        "gpu_launches": n_rep * K * m.launches_per_apply(),
        "roofline": {"bound": "hbm", "kernel": "probe_steer_team_kernel", "achieved": achieved, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": achieved / peaks["hbm_gbs"], "traffic": DECODE_DRAM_BYTES_PER_LAUNCH,
                     "traffic_source": "dram__bytes_read.sum + dram__bytes_write.sum of one launch of this kernel on this "
                                       "workload in an earlier ncu capture (not re-measured by this run)",
                     "frac_of_nominal_8000_gbs": achieved / NOMINAL_HBM_GBS,
                     "peak_source": peaks["source"],
                     "algorithmic_bytes_per_launch": nbytes,
                     "note": "2.9 MB per launch: launch-latency-bound by construction; the bandwidth- and tensor-bound "
                             "kernels of the other configs are in `targets`",
                     "protocol": {"steps_per_repeat": K, "repeats": n_rep, "timed_region_s": region_s,
                                  "ms_per_step": "median over timed passes of (pass time / steps in the pass)",
                                  "repeats_per_timed_pass": reps_per_pass, "us_per_step_over_passes": spread,
                                  "graph": "CUDA-graph replay; a graph launch holds %d consecutive steps (%d repeats of %d) over %d "
                                           "hidden buffers (%d MiB)" % (min(K, R) if K > R else R, reps_per_pass, K, R,
                                                                        R * T * d * 2 >> 20),
                                  "launch": "ordinary kernel launch (what a step costs behind any predecessor kernel)"},
                     "decode_step": {"probe_rows": rows_p, "steer_rows": rows_s,
                                     "us_added_per_decode_step": ms_per_step * 1e3,
                                     "us_added_per_decode_step_32_hooked_layers": 32 * ms_per_step * 1e3,
                                     "us_per_step_warm_l2": warm_us, "us_per_step_zero_live_rows": floor_us,
                                     "us_per_step_programmatic_launch_back_to_back": pdl_us,
                                     "status_word": status}},
    }
    if world == 1:
        line["cpu_baseline"] = cpu_baseline_block(args.cpu_seconds)
        if not args.no_extras:
            targets, ex = {}, {}
            try:
                collect_targets(targets, ex, w, hiddens, scores, peaks, mixlib, args)
            except Exception as e:                       # the other configs never break the contract line
                ex["error"] = repr(e)
            line["roofline"]["targets"] = targets
            line["extras"] = ex
    # the per-kernel detail first, the contract's own blocks last: whoever keeps only the end of a long line
    # keeps `roofline` (with `targets`) and `cpu_baseline`
    tail_keys = [k for k in ("clocks", "e2e", "gpu_launches", "cpu_baseline", "roofline") if k in line]
    line = {**{k: v for k, v in line.items() if k not in tail_keys}, **{k: line[k] for k in tail_keys}}
    print(json.dumps(line), flush=True)


def gpu_edit_hint(gi, sae, h_row):
    """Input recipe of configs 2 and 3 (outside every timed region): the features that fire on one row, so
    that half of a request's edits land on features it actually uses.  A plain torch product in row chunks."""
    x = h_row.float()
    z = torch.empty(sae.d_sae, dtype=torch.float32, device=x.device)
    for j0 in range(0, sae.d_sae, 8192):
        j1 = min(sae.d_sae, j0 + 8192)
        Wc = sae.W_enc[j0:j1]
        Wc = Wc.view(torch.float8_e4m3fn).float() * sae.w_scale[j0:j1, None] if sae.w_scale is not None else Wc.float()
        z[j0:j1] = Wc @ x + sae.b_enc[j0:j1]
    if sae.act == W.SAE_TOPK:
        top = torch.topk(z, sae.k)
        return top.indices[top.values > 0].cpu().numpy()
    thr = sae.theta if sae.theta is not None else torch.zeros_like(z)
    return torch.nonzero((z > thr) & (z > 0)).flatten().cpu().numpy()


def collect_targets(targets, ex, w, hiddens, scores, peaks, mixlib, args):
    """The other configurations: what the roofline targets are judged on goes to `targets` (compact), the
    per-kernel detail to `extras`."""
    sw = extras_sweep(peaks, mixlib)
    ex["sweep"] = sw
    targets["steer_stream"] = {"what": "steering alone, d=8192, T=65536 (2 GiB read + written)", "gbs": sw["steer"]["gbs"],
                               "frac_hbm": sw["steer"]["frac_hbm_peak"]}
    targets["probe_stream"] = {"what": "one-class probe alone, d=8192, T=65536 (1 GiB read)", "gbs": sw["probe"]["gbs"],
                               "frac_hbm": sw["probe"]["frac_hbm_peak"]}
    targets["encode_alone"] = {"what": sw["encode"]["shape"], "tflops": sw["encode"]["tflops"],
                               "frac_bf16_burst": sw["encode"]["frac_bf16_peak"]}
    tiny = extras_sae("tiny (config 0)", W.make_tiny("cuda"), peaks, mixlib)
    targets["cfg0_tiny"] = {"call_us": tiny["t_call_ms_graph"] * 1e3, "status": tiny["status"]}
    r2 = extras_sae("sae_heavy (config 2)", W.make_sae_heavy("cuda", edit_hint=gpu_edit_hint), peaks, mixlib)
    ex["sae_heavy"] = r2
    enc_ms = lambda r: max(r["stage_ms"]["encode"], r["stage_ms"].get("encode_pair", 0.0))
    targets["cfg2_sae_heavy"] = {"call_us": r2["t_call_ms_graph"] * 1e3, "encode_us": enc_ms(r2) * 1e3,
                                 "encode_w_enc_gbs": r2["encode_weight_stream_gbs"], "encode_frac_hbm": r2["encode_frac_hbm_peak"],
                                 "call_over_encode": r2["t_call_ms_graph"] / enc_ms(r2), "status": r2["status"]}
    torch.cuda.empty_cache()
    wm = W.make_mixed("cuda", edit_hint=gpu_edit_hint)
    r3 = extras_sae("mixed (config 3)", wm, peaks, mixlib)
    ex["mixed"] = r3
    targets["cfg3_mixed"] = {"call_us": r3["t_call_ms_graph"] * 1e3, "encode_us": enc_ms(r3) * 1e3,
                             "encode_tflops": r3["encode_tflops"], "encode_frac_bf16_burst": r3["encode_frac_bf16_peak"],
                             "encode_frac_bf16_sustained": r3["encode_frac_bf16_sustained"],
                             "call_over_encode": r3["t_call_ms_graph"] / enc_ms(r3), "status": r3["status"]}
    eo = extras_sae("mixed (config 3), edit-only shortcut", wm, peaks, mixlib, extra_flags=8)
    ex["mixed_edit_only_shortcut"] = {
        "note": "MIX_FLAG_SAE_EDIT_ONLY: JumpReLU rows with the error term skip the encode (16 dot products per row "
                "instead); an algorithmic shortcut, not counted toward any tensor-pipe fraction",
        "t_call_ms_graph": eo["t_call_ms_graph"], "stage_ms": eo["stage_ms"], "status": eo["status"]}
    del wm
    torch.cuda.empty_cache()
    rd = extras_replace_decode(peaks, mixlib)
    ex["replace_decode"] = rd
    targets["replace_decode"] = {"what": rd["what"], "decode_us": rd["decode_us"], "gather_gbs": rd["gather_gbs"],
                                 "frac_hbm": rd["frac_hbm_peak"], "status": rd["status"]}
    r4 = run_replay(peaks, mixlib, args.replays)
    ex["replay"] = r4
    targets["cfg4_replay"] = {"replays": r4["replays"], "bound_over_time": r4["bound_over_time"],
                              "t_call_ms": r4["t_call_ms"], "empty_replay_us": None if r4["empty_replay_ms"] is None else r4["empty_replay_ms"] * 1e3,
                              "n_live_covered": r4["n_live_covered"], "status_or": r4["status_or"]}
    torch.cuda.empty_cache()
    mc = extras_multiclass(peaks, mixlib)
    ex["multiclass_probes"] = mc
    targets["multiclass_probes"] = {
        "what": "whole call replayed from a graph, and the tensor-core probe kernel alone, as fractions of the HBM peak on hooked bytes",
        **{k: {"call_frac_hbm": round(v["graph_replay"]["frac_hbm_peak"], 3),
               "kernel_frac_hbm": round(v["probe_tc_kernel_alone"]["frac_hbm_peak"], 3), "status": v["status"]}
           for k, v in mc.items()}}
    ex["decode_variants"] = extras_decode_variants(w, hiddens[:256], scores[:256], mixlib)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="mix", choices=["mix", "reference"])
    ap.add_argument("--no-extras", action="store_true")
    ap.add_argument("--no-retile", action="store_true",
                    help="SAE contexts stream W_enc as registered instead of a tile-contiguous copy (MIX_FLAG_RETILE_W_ENC)")
    ap.add_argument("--workload", default="decode",
                    help="decode (the contract line) | sweep | sae_heavy | sae_heavy_fp8 | sae_heavy_fp8a | sae_small | sae_small_fp8 | sae_small_fp8a | mixed | mixed_fp8 | mixed_fp8a | mixed_edit_only | mixed_small | mixed_small_fp8a | conditional | conditional_small | replay_fp8 | replay_fp8a | multiclass | multiclass_small | replay")
    ap.add_argument("--cpu-seconds", type=float, default=8.0)
    ap.add_argument("--replays", type=int, default=60, help="replays of config 4 in the default run")
    args = ap.parse_args()
    if args.no_retile:
        global SAE_FLAGS
        SAE_FLAGS = 0
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank, world)
        return
    if args.workload != "decode":
        if rank == 0:
            run_workload(args)
        return
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local_rank)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    try:
        run_mix(args, rank, world, local_rank)
    finally:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of EliteKV decode attention on B200.

One step = one pass of the whole decode hot path for one layer over a batch of sequences:
    elitekv_append (1 new token per sequence) | elitekv_absorb_query -> elitekv_decode
(the append and the query preparation are independent and run on two streams).
Metric: decode-attention tokens/s (= sequences advanced per second for one layer), plus the
achieved cache-read bandwidth.  Workload at one GPU: LLaMA2-7B-shaped layer, 75 % KV reduction
(r = 8 elite chunks/head, d_c = 1536), batch 16, context 4096, contiguous cache, bf16,
synthetic seeded inputs.  With N GPUs every rank runs its own batch (sequences are
independent; no data-path collective) and the values add up.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

`--impl reference` times the float64 CPU oracle on a bounded sample of the same workload.
Prints one JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_01586_b200 import inputs as gen  # noqa: E402

METRIC = "decode_attention_tokens_per_s"
UNIT = "tokens/s"
NOMINAL_HBM_GBS = 8000.0


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# ---------------------------------------------------------------------------------------------
# clocks
# ---------------------------------------------------------------------------------------------
class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=self.tmp, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.tmp.flush()
        self.tmp.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.tmp.read().splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.tmp.close()
        try:
            os.unlink(self.tmp.name)
        except OSError:
            pass
        if sm:
            out["sm_mhz"] = statistics.median(sm)
            out["sm_max_mhz"] = max(mx)
        out["reasons"] = sorted(reasons)
        return out


# ---------------------------------------------------------------------------------------------
# CPU oracle leg
# ---------------------------------------------------------------------------------------------
def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def oracle_sample(w: gen.Workload, n_units: int, seed_shift: int = 0):
    """Times the oracle, as it stands, on `n_units` (sequence, head) units of the workload at
    full context: returns (seconds, units, description)."""
    from oracle import elitekv_oracle as O
    idx = gen.elite_index_sets(w).numpy().astype(np.int64)
    W_uk, W_uv = gen.up_projections(w, "cpu")
    W_uk, W_uv = W_uk.double().numpy(), W_uv.double().numpy()
    lens = gen.sequence_lengths(w).tolist()
    b = seed_shift % w.B
    n = int(lens[b])
    k_e, c = gen.tokens(w, n, "cpu", stream=1 + seed_shift)
    q = gen.queries(w, "cpu")[b].double().numpy()
    k_e, c = k_e.double().numpy(), c.double().numpy()
    heads = list(range(min(n_units, w.n_h)))
    t0 = time.perf_counter()
    O.decode_from_raw(q, n - 1, k_e, np.arange(n), c, W_uk, W_uv, idx, w.d_h, base=w.rope_base,
                      heads=heads)
    dt = time.perf_counter() - t0
    return dt, len(heads), f"{len(heads)} heads of sequence {b} at full context {n} (of {w.B}x{w.n_h} units)"


def cpu_baseline(w: gen.Workload, budget_s: float = 12.0):
    """Whole sequences (all heads) through the oracle until about `budget_s` seconds are spent."""
    t_total, units, seqs = 0.0, 0, 0
    while seqs < w.B and (seqs == 0 or t_total * (seqs + 1) / seqs < budget_s):
        dt, u, _ = oracle_sample(w, w.n_h, seed_shift=seqs)
        t_total += dt
        units += u
        seqs += 1
    value = (units / w.n_h) / t_total        # sequences (= decode tokens) per second, one layer
    return {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"{seqs} of {w.B} sequences, all {w.n_h} heads, full context; "
                      f"{t_total:.2f} s of oracle time"}


def config_of(w: gen.Workload, world: int):
    c = {"workload": w.name, "n_h": w.n_h, "d_h": w.d_h, "r": w.r, "d_c": w.d_c,
         "batch_per_gpu": w.B, "context": w.ctx, "paged": w.paged,
         "l2": "256 MiB flush write before every timed step; cache larger than L2",
         "parallelism": f"replicas x{world} (independent sequences, no collective)",
         "streams": "elitekv_decode_step: append + plan on the layer's second stream beside absorb_query; joined before the attention kernel"}
    return c


def run_reference(args, w: gen.Workload):
    """The oracle as it stands on the host cores: every step is one whole sequence of the
    workload (all heads, full context), the same sampling rule as `cpu_baseline`; a step of the
    workload advances B sequences, so ms_per_step is the measured time times B."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    times = []
    for i in range(args.warmup + args.steps):
        dt, u, what = oracle_sample(w, w.n_h, seed_shift=i)
        if i >= args.warmup:
            times.append(dt)
    per_seq = sum(times) / len(times)
    value = 1.0 / per_seq                # sequences (tokens) per second for one layer
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_seq * w.B * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": config_of(w, max(args.gpus, 1)),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                         "sample": f"each step one whole sequence (all {w.n_h} heads, full context) "
                                   f"of the {w.B}; ms_per_step is that time x {w.B}"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def max_over_ranks(dist, values, device):
    """Element-wise maximum of per-rank timings (ranks are independent replicas: the job is as
    slow as its slowest rank).  `dist` is torch.distributed or None for a single process."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.tolist()]


def aggregate_value(world: int, batch_per_rank: int, ms_per_step: float) -> float:
    """Whole-job decode tokens/s: every rank advances its own batch each step."""
    return world * batch_per_rank / (ms_per_step * 1e-3)


# ---------------------------------------------------------------------------------------------
# GPU leg
# ---------------------------------------------------------------------------------------------
def build_workload(w: gen.Workload, ek, device, decode_kernel: int = 0):
    """Cache prefilled with len-1 tokens per sequence; the step appends the last one."""
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, device)
    if w.d_ck:      # separated latents: B^k_S reads the first d_ck latent columns, B^v_S the rest
        W_uk, W_uv = W_uk[:w.d_ck].contiguous(), W_uv[w.d_ck:].contiguous()
    lens = gen.sequence_lengths(w)                       # tokens INCLUDING the decoded one
    B = w.B
    max_pos = int(lens.max()) + 1
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, max_pos, rope_base=w.rope_base,
                     decode_kernel=decode_kernel, d_ck=w.d_ck)
    rope_w = w.n_h * 2 * w.r
    page_table = None
    if w.paged:
        table, num_pages = gen.page_table(w, lens, headroom_tokens=0)
        rows, max_ctx = num_pages * w.page_size, 0
        page_table = table.to(device)
    else:
        max_ctx = int(lens.max())
        rows = B * max_ctx
    rope_plane = torch.zeros((rows, rope_w), dtype=torch.bfloat16, device=device)
    latent_plane = torch.zeros((rows, w.d_c), dtype=torch.bfloat16, device=device)
    cache = ek.make_cache(rope_plane, latent_plane, n_seqs=B, max_ctx=max_ctx,
                          page_table=page_table, page_size=w.page_size)
    # prefill through the library, sequence by sequence (bounded staging memory)
    for b in range(B):
        n = int(lens[b]) - 1
        if n <= 0:
            continue
        k_e, c = gen.tokens(w, n, device, stream=10 + b)
        seq = torch.full((n,), b, dtype=torch.int32, device=device)
        pos = torch.arange(n, dtype=torch.int32, device=device)
        ek.elitekv_append(layer, cache, k_e, c, seq, pos)
    torch.cuda.synchronize()
    # the step's inputs: one new token per sequence + the queries (host copies for the e2e leg)
    k_new, c_new = gen.tokens(w, B, "cpu", stream=5)
    q = gen.queries(w, "cpu")
    host = {
        "k_e": k_new.pin_memory(), "c": c_new.pin_memory(), "q": q.pin_memory(),
        "seq_id": torch.arange(B, dtype=torch.int32).pin_memory(),
        "pos": (lens - 1).to(torch.int32).pin_memory(),
        "lens": lens.to(torch.int32).pin_memory(),
    }
    dev = {k: v.to(device) for k, v in host.items()}
    ws = torch.empty(ek.elitekv_decode_workspace_size(layer, B), dtype=torch.uint8, device=device)
    bufs = {
        "q_rope": torch.empty((B, w.n_h, 2 * w.r), dtype=torch.bfloat16, device=device),
        "q_abs": torch.empty((B, w.n_h, layer.kw), dtype=torch.bfloat16, device=device),
        "out": torch.empty((B, w.n_h, w.d_h), dtype=torch.bfloat16, device=device),
        "out_host": torch.empty((B, w.n_h, w.d_h), dtype=torch.bfloat16).pin_memory(),
    }
    keep = (W_uk, W_uv, rope_plane, latent_plane, page_table)
    return layer, cache, lens, host, dev, ws, bufs, keep


def step(ek, layer, cache, d, ws, bufs):
    """One decode step through the library's single-call entry: the append and the work plan run
    on the layer's second stream beside the query preparation, joined before the attention."""
    ek.elitekv_decode_step(layer, cache, d["k_e"], d["c"], d["seq_id"], d["pos"], d["q"], d["lens"],
                           bufs["q_rope"], bufs["q_abs"], ws, bufs["out"])


KERNELS_PER_STEP = 5   # append, absorb, plan, split-K attention, combine + up-projection

SWEEP = ["7b-75pct-paged-b64-ragged", "13b-75pct-b32-ctx16384", "7b-50pct-b32-ctx8192",
         "7b-75pct-b32-ctx8192", "7b-87.5pct-b32-ctx8192", "7b-75pct-slrd512+1024-b32-ctx8192"]


def sweep_entry(ek, w: gen.Workload, device, flush, steps: int = 10, n_check: int = 2):
    """One of the other benchmark configurations: split-K kernel time and whole-step time on the
    device, plus the float64 oracle timed on `n_check` (sequence, head) units of the SAME inputs
    at full context (a cpu_baseline sample for this configuration) and the error of the library's
    output rows against those oracle rows."""
    layer, cache, lens, host, dev, ws, bufs, keep = build_workload(w, ek, device, 0)
    for _ in range(3):
        step(ek, layer, cache, dev, ws, bufs)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    for a, b in ev:
        flush.fill_(1)
        a.record()
        step(ek, layer, cache, dev, ws, bufs)
        b.record()
    torch.cuda.synchronize()
    step_ms = sum(a.elapsed_time(b) for a, b in ev) / steps
    ek.elitekv_profile_enable(layer, True)
    for _ in range(steps):
        flush.fill_(1)
        step(ek, layer, cache, dev, ws, bufs)
    torch.cuda.synchronize()
    kern_ms, kern_n = ek.elitekv_profile_collect(layer)
    ek.elitekv_profile_enable(layer, False)
    status = ek.elitekv_check_status(layer)
    cache_bytes = int(lens.sum()) * 2 * w.cache_elems_per_token
    kern_s = kern_ms / max(kern_n, 1) * 1e-3
    peak, peak_kind = measured_peaks()
    kernel_id = ek.elitekv_decode_plan_info(layer, cache, w.B)[0]
    out = bufs["out"].float().cpu().double().numpy()
    # ---- oracle on a few units of the same bytes
    from oracle import elitekv_oracle as O
    idx = gen.elite_index_sets(w).numpy().astype(np.int64)
    W_uk, W_uv = keep[0].double().cpu().numpy(), keep[1].double().cpu().numpy()
    g = np.random.default_rng(w.seed)
    t_cpu, num, den, mx = 0.0, 0.0, 0.0, 0.0
    for b in g.choice(w.B, size=min(n_check, w.B), replace=False).tolist():
        n = int(lens[b])
        k_e, c = gen.tokens(w, n - 1, device, stream=10 + b)
        k_e = torch.cat([k_e.cpu(), host["k_e"][b:b + 1]]).double().numpy()
        c = torch.cat([c.cpu(), host["c"][b:b + 1]]).double().numpy()
        h = int(g.integers(w.n_h))
        t0 = time.perf_counter()
        if w.d_ck:
            k_rope = O.rotate_elite_keys(k_e, np.arange(n), idx, w.d_h, w.rope_base)
            want = O.decode_slrd(host["q"][b].double().numpy(), n - 1, k_rope, c[:, :w.d_ck], c[:, w.d_ck:],
                                 W_uk, W_uv, idx, w.d_h, base=w.rope_base, heads=[h])[0]
        else:
            want = O.decode_from_raw(host["q"][b].double().numpy(), n - 1, k_e, np.arange(n), c, W_uk, W_uv,
                                     idx, w.d_h, base=w.rope_base, heads=[h])[0]
        t_cpu += time.perf_counter() - t0
        d = out[b, h] - want
        num += float(d @ d)
        den += float(want @ want)
        mx = max(mx, float(np.max(np.abs(d))))
    entry = {
        "workload": w.name, "kernel": kernel_id, "kernel_us": kern_s * 1e6,
        "achieved_gbs": cache_bytes / kern_s / 1e9, "frac": cache_bytes / kern_s / 1e9 / peak,
        "peak_kind": f"of {peak_kind}", "cache_bytes_per_step": cache_bytes, "ms_per_step": step_ms,
        "tokens_per_s": w.B / (step_ms * 1e-3), "status": status,
        "parity": {"units": n_check, "rel_l2": (num / den) ** 0.5 if den else None, "max_abs": mx},
        "cpu_baseline": {"value": 1.0 / (t_cpu / n_check * w.n_h), "unit": UNIT, "cores": oracle_threads(),
                         "kind": "oracle", "sample": f"{n_check} (sequence, head) units at full context, "
                                                     "scaled to all heads of a sequence"},
    }
    del layer, cache, dev, ws, bufs, keep
    torch.cuda.empty_cache()
    return entry


def project_append_bench(ek, device, flush, reps: int = 5):
    """The projection fused with the append (x [W^k_e, A^kv], 7B 75 % shape, d = 4096) at prefill
    size (T = 4096: tensor bound, bf16 TFLOP/s against the measured cuBLAS figure) and at the
    size of a decode batch (T = 16: bound by reading the 16.8 MB of weights once)."""
    w = gen.SWEEP_75
    d, T_max = 4096, 4096
    g = torch.Generator(device=device).manual_seed(4242)
    rope_w = w.n_h * 2 * w.r
    W_ke = (torch.randn(d, rope_w, generator=g, device=device) / d ** 0.5).to(torch.bfloat16)
    W_down = (torch.randn(d, w.d_c, generator=g, device=device) / d ** 0.5).to(torch.bfloat16)
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, device)
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, T_max + 1, W_ke=W_ke, W_down=W_down)
    rope_plane = torch.zeros((T_max, rope_w), dtype=torch.bfloat16, device=device)
    latent_plane = torch.zeros((T_max, w.d_c), dtype=torch.bfloat16, device=device)
    cache = ek.make_cache(rope_plane, latent_plane, n_seqs=1, max_ctx=T_max)
    x = torch.randn(T_max, d, generator=g, device=device).to(torch.bfloat16)
    seq = torch.zeros(T_max, dtype=torch.int32, device=device)
    pos = torch.arange(T_max, dtype=torch.int32, device=device)
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            tf_peak, tf_kind = float(json.load(f)["bf16_tflops"]), "of measured"
    except Exception:
        tf_peak, tf_kind = 1590.0, "of fallback"
    hbm_peak, hbm_kind = measured_peaks()
    out = {}
    for T in (T_max, 16):
        for _ in range(2):
            ek.elitekv_project_append(layer, cache, x[:T], seq[:T], pos[:T])
        evs = []
        for _ in range(reps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ek.elitekv_project_append(layer, cache, x[:T], seq[:T], pos[:T])
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        us = 1e3 * sum(a.elapsed_time(b) for a, b in evs) / reps
        flops = 2.0 * T * d * (rope_w + w.d_c)
        weight_bytes = 2 * d * (rope_w + w.d_c)
        out[f"T{T}"] = {"tokens": T, "us": us, "tflops": flops / (us * 1e-6) / 1e12,
                        "frac_tensor": flops / (us * 1e-6) / 1e12 / tf_peak, "tensor_peak_kind": tf_kind,
                        "weight_gbs": weight_bytes / (us * 1e-6) / 1e9,
                        "frac_hbm_weights": weight_bytes / (us * 1e-6) / 1e9 / hbm_peak, "hbm_peak_kind": f"of {hbm_kind}"}
    assert ek.elitekv_check_status(layer) == 0
    return out



def append_prefill(ek, device, flush, reps: int = 5):
    """Cache append at prefill size on the 7B 75 % shape: T = 4096 tokens of one sequence, and
    T = 32 x 4096 (a 4096-token prefill for each of 32 sequences).  Bytes = what the call must
    read plus what it must write, 2 x cache row bytes per token."""
    w = gen.SWEEP_75
    out = {}
    idx = gen.elite_index_sets(w)
    W_uk, W_uv = gen.up_projections(w, device)
    layer = ek.Layer(w.n_h, w.d_h, w.r, w.d_c, idx, W_uk, W_uv, 4096 + 1, rope_base=w.rope_base)
    peak, peak_kind = measured_peaks()
    for n_seq in (1, 32):
        T = n_seq * 4096
        rope_plane = torch.zeros((T, w.n_h * 2 * w.r), dtype=torch.bfloat16, device=device)
        latent_plane = torch.zeros((T, w.d_c), dtype=torch.bfloat16, device=device)
        cache = ek.make_cache(rope_plane, latent_plane, n_seqs=n_seq, max_ctx=4096)
        k_e, c = gen.tokens(w, T, device, stream=77)
        seq = torch.arange(n_seq, dtype=torch.int32, device=device).repeat_interleave(4096)
        pos = torch.arange(4096, dtype=torch.int32, device=device).repeat(n_seq)
        for _ in range(2):
            ek.elitekv_append(layer, cache, k_e, c, seq, pos)
        evs = []
        for _ in range(reps):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ek.elitekv_append(layer, cache, k_e, c, seq, pos)
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        us = 1e3 * sum(a.elapsed_time(b) for a, b in evs) / reps
        byts = 2 * T * 2 * w.cache_elems_per_token
        out[f"T{T}"] = {"tokens": T, "us": us, "bytes_read_plus_written": byts,
                        "gbs": byts / (us * 1e-6) / 1e9, "frac": byts / (us * 1e-6) / 1e9 / peak,
                        "peak_kind": f"of {peak_kind}"}
        del rope_plane, latent_plane, k_e, c, cache
        torch.cuda.empty_cache()
    assert ek.elitekv_check_status(layer) == 0
    return out




def attend_rows_bench(ek, layer, cache, w, lens, device, flush, cache_bytes, reps: int = 5):
    """m query rows per sequence over the bench workload's cache (causal; the rows sit at the last
    m positions): time of elitekv_attend_rows (plan + two-pass kernel + combine) and the cache
    bytes, counted ONCE, over that time.  Every row's block reads the whole tile, the first from
    HBM and the others from L2, so the ideal is still one pass over the cache."""
    peak, peak_kind = measured_peaks()
    out = {}
    lens_dev = lens.to(torch.int32).to(device)
    g = torch.Generator(device=device).manual_seed(99)
    for m in (2, 4, 8):
        try:
            q = torch.randn((w.B * m, w.n_h, w.d_h), generator=g, device=device).to(torch.bfloat16)
            q_pos = (lens_dev.view(-1, 1) - m + torch.arange(m, device=device, dtype=torch.int32).view(1, m))
            q_rope, q_abs = ek.elitekv_absorb_query(layer, q, q_pos.reshape(-1).to(torch.int32).contiguous())
            ws = torch.empty(ek.elitekv_attend_rows_workspace_size(layer, w.B, m), dtype=torch.uint8, device=device)
            res = torch.empty((w.B, m, w.n_h, w.d_h), dtype=torch.bfloat16, device=device)
            for _ in range(2):
                ek.elitekv_attend_rows(layer, cache, q_rope, q_abs, lens_dev, m, ws, res)
            evs = []
            for _ in range(reps):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                ek.elitekv_attend_rows(layer, cache, q_rope, q_abs, lens_dev, m, ws, res)
                b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            us = 1e3 * sum(a.elapsed_time(b) for a, b in evs) / reps
            out[f"m{m}"] = {"rows": m, "us": us, "query_rows_per_s": w.B * m / (us * 1e-6),
                            "cache_gbs_counted_once": cache_bytes / (us * 1e-6) / 1e9,
                            "frac": cache_bytes / (us * 1e-6) / 1e9 / peak, "peak_kind": f"of {peak_kind}"}
            del q, q_rope, q_abs, ws, res
        except ek.ElitekvError as exc:
            out[f"m{m}"] = {"rows": m, "skipped": str(exc)}
    assert ek.elitekv_check_status(layer) == 0
    return out


def ropelite_bench(ek, device, reps: int = 3):
    """RoPElite search (Algorithm 1) on synthetic activations of one 7B-shaped layer: 32 heads,
    d_h = 128, a calibration sequence of 2048 tokens, r = 8 rounds.  ALU-bound: per causal pair and
    chunk the kernel issues 9 FP32 lane instructions (two 2-term products, the rotated-minus-plain
    term, the masked residual sum, the absolute difference into the candidate's running sum);
    peak = SMs x 128 FP32 lanes x the maximum SM clock."""
    H, n, d_h, r = 32, 2048, 128, 8
    g = torch.Generator(device=device).manual_seed(31337)
    Q = torch.randn((H, n, d_h), generator=g, device=device).to(torch.bfloat16)
    K = torch.randn((H, n, d_h), generator=g, device=device).to(torch.bfloat16)
    ws = torch.empty(ek.elitekv_ropelite_workspace_size(H, n, d_h), dtype=torch.uint8, device=device)
    ek.elitekv_ropelite_search(Q, K, r, workspace=ws)
    evs = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        idx = ek.elitekv_ropelite_search(Q, K, r, workspace=ws)
        b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in evs) / reps
    pairs = H * n * (n + 1) // 2
    lane_instr = 9.0 * (d_h // 2) * pairs * r
    props = torch.cuda.get_device_properties(device)
    peak = props.multi_processor_count * 128 * 1.965e9
    # the float64 oracle on a small sample of the same activations: one head, 256 tokens, one round
    from oracle import ropelite_oracle as RO
    q64, k64 = Q[0, :256].double().cpu().numpy(), K[0, :256].double().cpu().numpy()
    t0 = time.perf_counter()
    want = RO.distances(q64, k64, [], d_h)
    t_cpu = time.perf_counter() - t0
    got = ek.elitekv_ropelite_distances(Q[:1, :256].contiguous(), K[:1, :256].contiguous())[0].double().cpu().numpy()
    return {"heads": H, "tokens": n, "d_h": d_h, "rounds": r, "ms": ms, "ms_per_round": ms / r,
            "head_rounds_per_s": H * r / (ms * 1e-3),
            "roofline": {"bound": "alu", "achieved": lane_instr / (ms * 1e-3) / 1e12, "peak": peak / 1e12,
                         "unit": "T FP32 lane-instr/s", "frac": lane_instr / (ms * 1e-3) / peak,
                         "peak_kind": "SMs x 128 lanes x 1965 MHz"},
            "parity_sample": {"rel_err_max": float(np.max(np.abs(got - want) / want))},
            "cpu_baseline": {"value": 1.0 / (t_cpu * (n * (n + 1) / 2) / (256 * 257 / 2)), "unit": "head-rounds/s",
                             "kind": "oracle", "cores": oracle_threads(),
                             "sample": "one head, 256 of 2048 tokens, one round; scaled by the number of causal pairs"},
            "first_head_elite": idx[0].tolist()}


def run_stage(args):
    from paper_2503_01586_b200 import binding as ek
    ek.lib()
    torch.cuda.set_device(0)
    device = torch.device("cuda", 0)
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=device)
    if args.stage == "append_prefill":
        rec = append_prefill(ek, device, flush, reps=2)
    elif args.stage == "project_append":
        rec = project_append_bench(ek, device, flush, reps=2)
    else:
        rec = ropelite_bench(ek, device, reps=1)
    print(json.dumps({"stage": args.stage, "record": rec}))


def run_gpu(args, w: gen.Workload):
    from paper_2503_01586_b200 import binding as ek
    ek.lib()   # fail loudly if the CUDA library is missing
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    device = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist_mod.init_process_group("nccl", device_id=device)
        dist = dist_mod

    w_rank = gen.replace(w, seed=w.seed + 100 * rank) if rank else w
    layer, cache, lens, host, dev, ws, bufs, keep = build_workload(w_rank, ek, device, args.kernel)
    total_tokens = int(lens.sum())
    bytes_per_token = 2 * w.cache_elems_per_token
    cache_bytes = total_tokens * bytes_per_token
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device=device)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    sampler = ClockSampler(local) if rank == 0 else None
    for _ in range(max(args.warmup, 3)):
        step(ek, layer, cache, dev, ws, bufs)
    torch.cuda.synchronize()
    assert ek.elitekv_check_status(layer) == 0

    # ---- device-resident timing: K steps, L2 flushed before each, events around each step
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    barrier()
    for a, b in ev:
        flush.fill_(1)
        a.record()
        step(ek, layer, cache, dev, ws, bufs)
        b.record()
    barrier()
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = sum(step_ms)
    # ---- the same K steps again with the library's event pair around the split-K kernel (kept
    #      out of the timed steps above: an event record between two launches holds back the
    #      programmatic overlap of their prologues)
    ek.elitekv_profile_enable(layer, True)
    for _ in range(args.steps):
        flush.fill_(1)
        step(ek, layer, cache, dev, ws, bufs)
    torch.cuda.synchronize()
    kern_ms, kern_n = ek.elitekv_profile_collect(layer)
    ek.elitekv_profile_enable(layer, False)

    # ---- end to end: host buffers in, host result out, every step, through the library's step
    #      runner: the six small input arrays live in ONE pinned staging buffer and cross in one
    #      copy, the step runs, the result is copied back and the host waits for it.  The headline
    #      replays the runner's CUDA graph (what a serving loop does); the eager number (same
    #      work enqueued call by call, bound by host launch latency) is reported beside it.
    def e2e_time(runner):
        for k in runner.ORDER:
            runner.host[k].copy_(host[k].view(runner.host[k].shape))
        for _ in range(3):
            runner.run()
        assert torch.equal(runner.out_host, bufs["out"].cpu())      # same step, same bits
        barrier()
        t0 = time.perf_counter()
        for _ in range(args.steps):
            runner.run()         # no flush here: the 268 MB+ cache does not fit the 126 MB L2
        torch.cuda.synchronize()
        return time.perf_counter() - t0

    eager_runner = ek.DecodeStepRunner(layer, cache, w.B, device, graph=False)
    h2d, d2h = eager_runner.h2d_bytes, eager_runner.d2h_bytes
    e2e_eager_s = e2e_time(eager_runner)
    e2e_mode = "cuda graph replay (DecodeStepRunner)"
    try:
        e2e_s = e2e_time(ek.DecodeStepRunner(layer, cache, w.B, device, graph=True))
    except Exception as exc:      # capture not possible in this environment: the eager number stands
        print(f"[bench] CUDA-graph end-to-end leg failed, reporting the eager one: {exc}", file=sys.stderr)
        e2e_s, e2e_mode = e2e_eager_s, "eager (DecodeStepRunner, graph capture failed)"
    assert ek.elitekv_check_status(layer) == 0

    # ---- per-call breakdown (informational; same kernels, a few extra untimed-by-the-metric calls)
    def timed(fn, n=10):
        evs = []
        for _ in range(n):
            flush.fill_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            evs.append((a, b))
        torch.cuda.synchronize()
        return 1e3 * sum(a.elapsed_time(b) for a, b in evs) / n
    stages = {
        "append_us": timed(lambda: ek.elitekv_append(layer, cache, dev["k_e"], dev["c"], dev["seq_id"], dev["pos"])),
        "absorb_us": timed(lambda: ek.elitekv_absorb_query(layer, dev["q"], dev["pos"], bufs["q_rope"], bufs["q_abs"])),
        "decode_us": timed(lambda: ek.elitekv_decode(layer, cache, bufs["q_rope"], bufs["q_abs"], dev["lens"], ws, bufs["out"])),
    }
    # keep the GPU busy long enough for the clock sampler to see it under load
    t_busy = time.perf_counter()
    while time.perf_counter() - t_busy < 0.6:
        for _ in range(20):
            step(ek, layer, cache, dev, ws, bufs)
        torch.cuda.synchronize()
    clocks = sampler.stop() if sampler else None
    assert ek.elitekv_check_status(layer) == 0

    # ---- comparator: uncompressed RoPE-MHA decode at the same shape (rank 0, one GPU)
    comparator = None
    if rank == 0 and not w.paged and not args.no_comparator:
        try:
            max_ctx = int(lens.max())
            K, V = gen.mha_cache(w, w.B * max_ctx, device)
            K = K.view(w.B, max_ctx, w.n_h, w.d_h)
            V = V.view(w.B, max_ctx, w.n_h, w.d_h)
            qh = dev["q"]
            mws = torch.empty(ek.elitekv_mha_workspace_size(w.B, w.n_h, w.d_h), dtype=torch.uint8,
                              device=device)
            mo = torch.empty_like(qh)
            for _ in range(3):
                ek.elitekv_mha_decode(qh, K, V, dev["lens"], mws, mo)
            evs = []
            for _ in range(min(args.steps, 20)):
                flush.fill_(1)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record()
                ek.elitekv_mha_decode(qh, K, V, dev["lens"], mws, mo)
                b.record()
                evs.append((a, b))
            torch.cuda.synchronize()
            ms = sum(a.elapsed_time(b) for a, b in evs) / len(evs)
            mha_bytes = total_tokens * 4 * w.n_h * w.d_h
            comparator = {"kind": "uncompressed RoPE-MHA decode, same shape", "ms": ms,
                          "tokens_per_s": w.B / (ms * 1e-3), "cache_bytes": mha_bytes,
                          "gbs": mha_bytes / (ms * 1e-3) / 1e9}
            del K, V
        except torch.cuda.OutOfMemoryError:
            comparator = None

    # ---- the other benchmark configurations and the prefill append (one GPU, rank 0 only)
    sweep, prefill, projection, rows, ropelite = None, None, None, None, None
    if rank == 0 and world == 1 and not args.no_sweep:
        rows = attend_rows_bench(ek, layer, cache, w, lens, device, flush, cache_bytes)
        del layer, cache, dev, ws, bufs, keep, eager_runner
        torch.cuda.empty_cache()
        t_sweep = time.perf_counter()
        prefill = append_prefill(ek, device, flush)
        projection = project_append_bench(ek, device, flush)
        ropelite = ropelite_bench(ek, device)
        sweep = []
        for name in SWEEP:
            if name == w.name:
                continue
            if time.perf_counter() - t_sweep > args.sweep_budget_s:
                sweep.append({"workload": name, "skipped": "sweep time budget spent"})
                continue
            try:
                sweep.append(sweep_entry(ek, gen.CONFIGS[name], device, flush))
            except torch.cuda.OutOfMemoryError:
                sweep.append({"workload": name, "skipped": "out of device memory"})
                torch.cuda.empty_cache()

    # ---- reduce over ranks
    total_ms, e2e_s, kern_ms = max_over_ranks(dist, [total_ms, e2e_s, kern_ms], device)
    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    ms_per_step = total_ms / args.steps
    value = aggregate_value(world, w.B, ms_per_step)
    kern_avg_s = (kern_ms / max(kern_n, 1)) * 1e-3
    achieved = cache_bytes / kern_avg_s / 1e9 if kern_n else None
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": config_of(w, world),
        "cache_bytes_per_step": cache_bytes,
        "hbm_gbs_whole_step": cache_bytes / (ms_per_step * 1e-3) / 1e9,
        "pct_of_nominal_8tbs_whole_step": 100.0 * cache_bytes / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS,
        "roofline": {"bound": "hbm", "kernel": "split-K decode attention", "achieved": achieved,
                     "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                     "frac": (achieved / peak) if achieved else None,
                     "frac_of_nominal_8tbs": (achieved / NOMINAL_HBM_GBS) if achieved else None,
                     "kernel_us": kern_avg_s * 1e6, "launches_timed": kern_n,
                     "traffic": TRAFFIC_BYTES_PER_LAUNCH.get(w.name)},
        "e2e": {"value": world * w.B * args.steps / e2e_s, "unit": UNIT,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "mode": e2e_mode,
                "value_eager": world * w.B * args.steps / e2e_eager_s},
        "gpu_launches": KERNELS_PER_STEP * args.steps,
        "clocks": clocks,
        "stages": stages,
        "comparator": comparator,
    }
    if not args.no_cpu_baseline and world == 1:
        line["cpu_baseline"] = cpu_baseline(w)
    else:
        line["cpu_baseline"] = None
    line["stages"]["append_prefill"] = prefill
    line["stages"]["project_append"] = projection
    line["stages"]["attend_rows"] = rows
    line["stages"]["ropelite_search"] = ropelite
    line["sweep"] = sweep
    print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


# dram__bytes_read.sum + dram__bytes_write.sum of one split-K launch on the named workload, from an
# ncu capture of the kernel that serves it (None where no capture of the current kernel exists).
TRAFFIC_BYTES_PER_LAUNCH = {
    "7b-75pct-b16-ctx4096": 270263040 + 4182528,     # resident-tile kernel, one launch
}


def run_dry(args, w: gen.Workload):
    """The multi-rank plumbing of the GPU leg on CPU: rank environment, process group (gloo),
    barrier, max over ranks, aggregate value, one JSON line from rank 0."""
    import torch.distributed as dist
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world > 1:
        dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = 1.0 + rank                         # the slowest rank decides
    (ms_max,) = max_over_ranks(dist if world > 1 else None, [ms], "cpu")
    if rank == 0:
        print(json.dumps({"metric": METRIC, "n_gpus": world, "ms_per_step": ms_max,
                          "value": aggregate_value(world, w.B, ms_max), "dry_run": True}))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def launch_replicas(args) -> int:
    """`bench.py --gpus N` started plainly (no torchrun): starts N copies of this script, one per
    GPU, each with the rank environment torchrun would give it; rank 0 prints the JSON line.
    Fails loudly when the machine has fewer than N devices or a replica fails."""
    import socket
    n = args.gpus
    if args.impl != "reference" and not args.dry_run_ranks:
        have = torch.cuda.device_count()
        if have < n:
            raise SystemExit(f"bench.py --gpus {n}: only {have} CUDA device(s) visible")
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    procs = []
    for r in range(n):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    codes = [p.wait() for p in procs]
    if any(codes):
        raise SystemExit(f"bench.py --gpus {n}: replica exit codes {codes}")
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=gen.LLAMA7B_75.name, choices=sorted(gen.CONFIGS))
    ap.add_argument("--kernel", type=int, default=0,
                    help="split-K kernel: 0 auto, 1 CUDA-core, 2 tcgen05 two-pass, 3 tcgen05 resident tile")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-comparator", action="store_true")
    ap.add_argument("--no-sweep", action="store_true",
                    help="skip the other configurations and the prefill-append measurement")
    ap.add_argument("--sweep-budget-s", type=float, default=150.0)
    ap.add_argument("--dry-run-ranks", action="store_true",
                    help="launcher check without a GPU: every rank joins a gloo group, takes part in the "
                         "max-over-ranks reduction of a dummy timing and rank 0 prints a JSON line")
    ap.add_argument("--stage", default=None, choices=["append_prefill", "project_append", "ropelite_search"],
                    help="time only this side measurement and print its record (for profiling one kernel)")
    args = ap.parse_args()
    w = gen.CONFIGS[args.workload]
    if args.stage:
        run_stage(args)
        return
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        launch_replicas(args)
        return
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world != max(args.gpus, 1):
        raise SystemExit(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}")
    if args.dry_run_ranks:
        run_dry(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_gpu(args, w)


if __name__ == "__main__":
    main()

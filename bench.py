#!/usr/bin/env python
"""Benchmark of the chunk-attention hot path (plan -> KV append -> tile + streaming attention -> merge).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole path over one synthetic batch: one hat_chunk_attention call with the
append fused (for the multi-call workloads, the whole sequence of calls).  Prints ONE JSON line.
With N > 1 (torchrun) every rank runs an independent replica of the batch (the path has no
inter-GPU exchange); time is the maximum over ranks and the value sums the work of all ranks.
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

from paper_2503_18989_b200 import workloads as W  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
VERIFY_MAX_ROWS = 16          # chunks up to this length take the streaming kernel
SLOT_NAMES = ["kv_append", "tile_attention", "streaming_attention", "merge"]


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"]))}, "measured"
    except Exception:
        return dict(FALLBACK_PEAKS), "fallback"


# ----------------------------------------------------------------------------
# algorithmic work of a batch (conventions: only unmasked (q,k) pairs, 2d flop for QK^T + 2d for PV;
# every visible K and V row read once per head)
# ----------------------------------------------------------------------------
def step_work(cache, st):
    Hkv, d, e = cache.num_heads, cache.head_dim, 2
    H = int(st.q.shape[1])                      # query heads (= K/V heads in the paper's models)
    P = st.prefix_len.astype(np.int64)
    Cn = st.chunk_len.astype(np.int64)
    pairs = Cn * P + Cn * (Cn + 1) // 2         # causal count, also when a token tree thins the chunk's own keys
    flops = 4 * d * H * pairs
    kv_bytes = 2 * (P + Cn) * Hkv * d * e * (Cn > 0)
    io_bytes = Cn * H * d * e + Cn * H * d * 4 + Cn * H * 4            # q in, out + lse out
    short = (Cn > 0) & (Cn <= VERIFY_MAX_ROWS)
    long_ = Cn > VERIFY_MAX_ROWS
    T = int(Cn.sum())
    return {
        "flops": int(flops.sum()),
        "tile_flops": int(flops[long_].sum()), "tile_bytes": int((kv_bytes + io_bytes)[long_].sum()),
        "stream_flops": int(flops[short].sum()), "stream_bytes": int((kv_bytes + io_bytes)[short].sum()),
        "append_bytes": int(4 * T * Hkv * d * e),
        "kv_bytes": int(kv_bytes.sum()),
        "rows": T,
    }


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.samples = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None
            return
        threading.Thread(target=self._pump, daemon=True).start()

    def _pump(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0, t1):
        inside = [s for s in self.samples if t0 <= s[0] <= t1]
        pool = inside or self.samples[-3:]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for _, line in pool:
            f = [x.strip() for x in line.split(",")]
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except Exception:
                continue
            for name, val in zip(names, f[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(inside)}


# ----------------------------------------------------------------------------
# replicas: the path has no inter-GPU exchange, so N ranks run N independent copies of the batch
# ----------------------------------------------------------------------------
def replica_seed(workload: str, rank: int) -> int:
    """Seed of rank `rank`'s replica: the workload's own seed for rank 0, shifted by 1000 per rank."""
    return W.SEED_BASE + list(W.WORKLOADS).index(workload) + 1 + 1000 * rank


def max_over_ranks(values, world: int, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity when world == 1)."""
    if world <= 1:
        return [float(v) for v in values]
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def whole_job_value(flops_per_replica_step: int, world: int, ms_per_step: float) -> float:
    """TFLOP/s of the whole job: every rank does the same amount of work in the (max-over-ranks) step time."""
    return world * flops_per_replica_step / (ms_per_step * 1e-3) / 1e12


NOMINAL = {"tensor_tflops": 2250.0, "hbm_gbs": 8000.0}      # dense 16-bit tensor peak and HBM3e bandwidth of a B200, nominal


def pick_tensor_peak(peaks, peak_kind, timed_seconds, reasons):
    """Denominator for a tensor-bound kernel: the burst figure when the timed region is well under a second and the
    sampled clocks show no power cap (a kernel timed alone), else the sustained one (a kernel inside a long loop)."""
    burst = timed_seconds < 1.0 and "sw_power_cap" not in (reasons or [])
    key = "bf16_tflops" if burst else "bf16_tflops_sustained"
    return peaks[key], f"{peak_kind} bf16 {'burst' if burst else 'sustained'}"


def kernel_table(total, works, n_calls, kernel_ms, kernel_calls, peaks, tensor_peak):
    """Per kernel: achieved algorithmic throughput from its mean CUDA-event duration, against every denominator."""
    avg = np.where(kernel_calls > 0, kernel_ms / np.maximum(kernel_calls, 1), 0.0)   # ms per launch
    per_launch = {
        "kv_append": ("hbm", total["append_bytes"] / n_calls),
        "tile_attention": ("tensor", total["tile_flops"] / max(1, sum(1 for w in works if w["tile_flops"]))),
        "streaming_attention": ("hbm", total["stream_bytes"] / max(1, sum(1 for w in works if w["stream_bytes"]))),
        "merge": ("hbm", 0.0),
    }
    kernels = {}
    for i, name in enumerate(SLOT_NAMES):
        if kernel_calls[i] == 0:
            continue
        bound, alg = per_launch[name]
        sec = avg[i] * 1e-3
        if bound == "tensor":
            ach, peak, unit = alg / sec / 1e12, tensor_peak, "TFLOP/s"
            extra = {"frac_burst": ach / peaks["bf16_tflops"], "frac_sustained": ach / peaks["bf16_tflops_sustained"],
                     "frac_nominal": ach / NOMINAL["tensor_tflops"]}
        else:
            ach, peak, unit = alg / sec / 1e9, peaks["hbm_gbs"], "GB/s"
            extra = {"frac_nominal": ach / NOMINAL["hbm_gbs"]}
            if ach > peak:
                extra["note"] = "above 1: the denominator is a measured COPY (read + write); a read-only stream can exceed it"
        kernels[name] = {"bound": bound, "achieved": ach, "peak": peak, "unit": unit, "frac": ach / peak, **extra,
                         "ms_per_launch": float(avg[i]), "launches": int(kernel_calls[i]),
                         "share": float(kernel_ms[i] / max(kernel_ms.sum(), 1e-9))}
    if "tile_attention" in kernels:
        # the tile kernel against the memory roofline as well (short chunks are HBM-bound)
        sec = kernels["tile_attention"]["ms_per_launch"] * 1e-3
        n_tile_calls = max(1, sum(1 for w in works if w["tile_flops"]))
        kernels["tile_attention"]["algorithmic_bytes"] = int(total["tile_bytes"] / n_tile_calls)
        kernels["tile_attention"]["hbm_gbs"] = total["tile_bytes"] / n_tile_calls / sec / 1e9
        kernels["tile_attention"]["hbm_frac"] = kernels["tile_attention"]["hbm_gbs"] / peaks["hbm_gbs"]
    return kernels


def step_bound(total, ms_per_step, peaks, tensor_peak):
    """Roofline of the whole step: T_roof = max(F / pi, B / beta) over all algorithmic flops and bytes (K/V read once
    per head, q in, out + lse out, append read + write), measured and nominal peaks."""
    F = total["flops"]
    Bt = total["tile_bytes"] + total["stream_bytes"] + total["append_bytes"]
    t_meas = max(F / (tensor_peak * 1e12), Bt / (peaks["hbm_gbs"] * 1e9)) * 1e3
    t_nom = max(F / (NOMINAL["tensor_tflops"] * 1e12), Bt / (NOMINAL["hbm_gbs"] * 1e9)) * 1e3
    return {"flops": int(F), "bytes": int(Bt), "t_roof_ms": t_meas, "step_frac": t_meas / ms_per_step,
            "t_roof_nominal_ms": t_nom, "step_frac_nominal": t_nom / ms_per_step,
            "flops_over_peak_ms": F / (tensor_peak * 1e12) * 1e3, "bytes_over_bandwidth_ms": Bt / (peaks["hbm_gbs"] * 1e9) * 1e3}


def quick_config(name, device, stream, peaks, peak_kind, K=20, warmup=3, with_oracle=True, samples=96):
    """One of the named workloads, briefly: K timed steps (L2 flushed where the K/V working set would fit in it),
    per-kernel roofline figures, and the largest deviation from the CPU oracle on sampled (request, row, head) triples
    of the last call."""
    import torch
    from paper_2503_18989_b200 import binding as B
    from paper_2503_18989_b200 import runner
    sc = W.WORKLOADS[name]()
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, device)
    steps = [runner.DeviceStep(cache, st) for st in sc.steps]
    works = [step_work(sc.cache, st) for st in sc.steps]
    total = {k: sum(w[k] for w in works) for k in works[0]}
    flush_l2 = total["kv_bytes"] / len(sc.steps) < 2 * L2_BYTES
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device) if flush_l2 else None

    def one_step():
        for ds in steps:
            ds.attend(fused_append=True, stream=stream)
    for _ in range(warmup):
        one_step()
    torch.cuda.synchronize(device)
    for ds in steps:
        B.hat_plan_enable_timing(ds.plan, K)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in evs:
        if flush_l2:
            flush_buf.zero_()
        a.record(); one_step(); b.record()
    torch.cuda.synchronize(device)
    elapsed_ms = sum(a.elapsed_time(b) for a, b in evs)
    kernel_ms = np.zeros(B.HAT_TIMING_SLOTS)
    kernel_calls = np.zeros(B.HAT_TIMING_SLOTS)
    for ds in steps:
        ms = B.hat_plan_read_timing(ds.plan, K)
        kernel_ms += ms.sum(axis=0)
        kernel_calls += (ms > 0).sum(axis=0)
    status = [B.hat_last_device_status(ds.plan, stream) for ds in steps]
    ms_per_step = elapsed_ms / K
    tensor_peak, source = pick_tensor_peak(peaks, peak_kind, elapsed_ms * 1e-3, [])
    res = {"ms_per_step": ms_per_step, "steps": K, "calls_per_step": len(sc.steps), "dtype": sc.cache.dtype,
           "l2": "flushed between steps" if flush_l2 else "KV working set larger than L2",
           "value_tflops": total["flops"] / (ms_per_step * 1e-3) / 1e12,
           "kv_gbs": total["kv_bytes"] / (ms_per_step * 1e-3) / 1e9, "tensor_peak_source": source,
           "kernels": kernel_table(total, works, len(sc.steps), kernel_ms, kernel_calls, peaks, tensor_peak),
           "step_roofline": step_bound(total, ms_per_step, peaks, tensor_peak),
           "device_status_ok": all(s == B.HAT_OK for s in status)}
    if with_oracle:
        from oracle import hat_oracle as O
        st = sc.steps[-1]
        out, lse = steps[-1].results()
        kp, vp = cache.pools_to_host()                # the GPU's own pools after the appends (checked bit for bit in tests/)
        rng = np.random.default_rng(1)
        live = np.nonzero(st.chunk_len > 0)[0]
        tri = np.asarray([(r, int(rng.integers(st.chunk_len[r])), int(rng.integers(st.q.shape[1])))
                          for r in live[rng.integers(len(live), size=samples)]], np.int64)
        wo, wl = O.attention_rows(sc.cache, kp, vp, st, tri)
        rows = st.cu_chunk[tri[:, 0]] + tri[:, 1]
        res["oracle_sample"] = {"triples": int(len(tri)),
                                "max_abs_out": float(np.abs(out[rows, tri[:, 2]].astype(np.float64) - wo).max()),
                                "max_abs_lse": float(np.abs(lse[rows, tri[:, 2]].astype(np.float64) - wl).max())}
    for ds in steps:
        ds.close()
    del steps, cache, flush_buf
    torch.cuda.empty_cache()
    return res


def layer_front(sc, cache, ds, device, stream, peaks, peak_kind, K=20, warmup=3, with_oracle=True):
    """The step in front of the attention module for the first call of the workload (Sec. 2.1: Q = X W_Q, K = X W_K,
    V = X W_V): the projection kernel with the rotation and the cache write in its epilogue, hidden = heads x head_dim.
    K timed launches with the L2 flushed in between; a few rows against the float64 oracle."""
    import torch
    from paper_2503_18989_b200 import binding as B
    from paper_2503_18989_b200 import runner
    st = sc.steps[0]
    spec = sc.cache
    hq, hkv, d = int(st.q.shape[1]), spec.num_heads, spec.head_dim
    hidden, feats, T = hq * d, (hq + 2 * hkv) * d, st.total_rows
    xb, wb = W.projection_inputs(900, spec.dtype, T, hidden, feats)
    x_dev, w_dev = runner._dev_u16(xb, device), runner._dev_u16(wb, device)
    q_out = torch.empty((T, hq, d), dtype=torch.int16, device=device)
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device)
    launches0 = B.hat_launch_count()
    for _ in range(warmup):
        B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q_out, 10000.0, False, stream)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    for a, b in evs:
        flush_buf.zero_()
        a.record()
        B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q_out, 10000.0, False, stream)
        b.record()
    torch.cuda.synchronize(device)
    ms = float(np.median([a.elapsed_time(b) for a, b in evs]))
    flops = 2.0 * T * hidden * feats
    tensor_peak, source = pick_tensor_peak(peaks, peak_kind, K * ms * 1e-3, [])
    e = 2
    res = {"op": "qkv projection + rotation + cache write (hat_qkv_rope_append)", "rows": T, "hidden": hidden,
           "features": feats, "dtype": spec.dtype, "ms": ms, "tflops": flops / (ms * 1e-3) / 1e12,
           "bound": "tensor", "peak": tensor_peak, "peak_source": source,
           "frac": flops / (ms * 1e-3) / 1e12 / tensor_peak,
           "frac_nominal": flops / (ms * 1e-3) / 1e12 / NOMINAL["tensor_tflops"],
           "algorithmic_bytes": (T * hidden + feats * hidden + T * feats) * e,
           "launches": (B.hat_launch_count() - launches0) // (warmup + K),
           "device_status_ok": B.hat_last_device_status(ds.plan, stream) == B.HAT_OK}
    # the attention step on the projection's own q rows and on the cache it wrote: no append kernel, no k_new / v_new
    # read (the projection's cache write stands in for it), timed as projection + attention back to back
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
           for _ in range(K)]
    for a, m, b in evs:
        flush_buf.zero_()
        a.record()
        B.hat_qkv_rope_append(cache.desc, ds.plan, x_dev, hidden, w_dev, q_out, 10000.0, False, stream)
        m.record()
        B.hat_chunk_attention(cache.desc, ds.plan, q_out, None, None, ds.out, ds.lse, 0.0, ds.workspace,
                              ds.workspace_bytes, stream)
        b.record()
    torch.cuda.synchronize(device)
    res["then_attention_without_append_ms"] = float(np.median([m.elapsed_time(b) for a, m, b in evs]))
    res["projection_and_attention_ms"] = float(np.median([a.elapsed_time(b) for a, m, b in evs]))
    res["device_status_ok"] = res["device_status_ok"] and B.hat_last_device_status(ds.plan, stream) == B.HAT_OK
    if with_oracle:
        from oracle import hat_qkv_oracle as QO
        from oracle import hat_rope_oracle as RO
        rows = np.unique(np.random.default_rng(2).integers(0, T, size=16))
        pos = RO.positions(st)
        want_q, _, _ = QO.qkv_rope(xb[rows], wb, pos[rows], spec.dtype, hq, hkv, d)
        got_q = q_out[torch.from_numpy(rows).to(device)].cpu().numpy().view(np.uint16)
        gw, ww = W.bits_to_f64(got_q, spec.dtype), W.bits_to_f64(want_q, spec.dtype)
        res["oracle_sample"] = {"rows": int(len(rows)), "same_bits_share": float(np.mean(got_q == want_q)),
                                "max_abs_q": float(np.abs(gw - ww).max())}
    del x_dev, w_dev, q_out, flush_buf
    torch.cuda.empty_cache()
    return res


def lookup_traffic(kernel: str, workload: str):
    """DRAM bytes per launch from the committed ncu capture of this kernel on this workload, or None when
    there is none or the kernel source has changed since (profiles/traffic.json records a source hash)."""
    import hashlib
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            table = json.load(f)["entries"]
        for e in table:
            if e["kernel"] == kernel and e["workload"] == workload:
                with open(os.path.join(ROOT, e["source"]), "rb") as src:
                    if hashlib.sha256(src.read()).hexdigest()[:16] == e["source_sha256_16"]:
                        return int(e["traffic_bytes"])
    except Exception:
        pass
    return None


def pick_oracle_sample(cache, st, rng, target_flops):
    """(request, row, head) units drawn uniformly over all (row, head) pairs until ~target_flops."""
    H, d = int(st.q.shape[1]), cache.head_dim
    live = np.nonzero(st.chunk_len > 0)[0]
    rows_req = np.repeat(live, st.chunk_len[live])
    rows_i = np.concatenate([np.arange(int(st.chunk_len[r])) for r in live])
    units, flops = [], 0
    while flops < target_flops and len(units) < 200000:
        t = int(rng.integers(len(rows_req)))
        r, i, h = int(rows_req[t]), int(rows_i[t]), int(rng.integers(H))
        units.append((r, i, h))
        flops += 4 * d * (int(st.prefix_len[r]) + i + 1)
    return np.asarray(units, np.int64), flops


def time_oracle(sc, budget_s, seed=0):
    """The CPU oracle on a bounded sample of the last call of the workload.  Returns
    (flop/s, cores, description, units, flops_per_run)."""
    from oracle import hat_oracle as O
    st = sc.steps[-1]
    kp, vp = sc.k_pool, sc.v_pool
    for s in sc.steps:                       # the oracle needs the chunk's K/V in its pool (append, then attend)
        O.kv_append(sc.cache, kp, vp, s)
    rng = np.random.default_rng(seed)
    units, fl = pick_oracle_sample(sc.cache, st, rng, 2e8)
    t0 = time.perf_counter(); O.attention_rows(sc.cache, kp, vp, st, units); dt = time.perf_counter() - t0
    rate = fl / max(dt, 1e-6)
    units, fl = pick_oracle_sample(sc.cache, st, rng, rate * budget_s)
    t0 = time.perf_counter(); O.attention_rows(sc.cache, kp, vp, st, units); dt = time.perf_counter() - t0
    return fl / dt, O.threads(), f"{len(units)} (request,row,head) units of the batch, {fl:.3g} flop, {dt:.1f} s", \
        units, fl


def make_workload(args, seed=None):
    """The named workload; --q-group / --tree reach the two workloads that have decode-phase requests."""
    kw = {} if seed is None else {"seed": seed}
    if args.q_group != 1 or args.tree:
        if args.workload not in ("spec_verify", "mixed_13b"):
            raise SystemExit("--q-group and --tree apply to spec_verify and mixed_13b only")
        kw.update(q_group=args.q_group, tree=args.tree)
    return W.WORKLOADS[args.workload](**kw)


def run_reference(args, rank):
    """Reference arm: the CPU oracle, as it stands, on the host cores."""
    if rank != 0:
        return
    from oracle import hat_oracle as O
    sc = make_workload(args)
    st = sc.steps[-1]
    for s in sc.steps:
        O.kv_append(sc.cache, sc.k_pool, sc.v_pool, s)
    rng = np.random.default_rng(0)
    units, fl = pick_oracle_sample(sc.cache, st, rng, 2e8)
    t0 = time.perf_counter(); O.attention_rows(sc.cache, sc.k_pool, sc.v_pool, st, units)
    rate = fl / max(time.perf_counter() - t0, 1e-6)
    per_step = min(20.0, args.cpu_budget, 150.0 / max(1, args.steps + args.warmup))
    units, fl = pick_oracle_sample(sc.cache, st, rng, rate * per_step)
    for _ in range(args.warmup):
        O.attention_rows(sc.cache, sc.k_pool, sc.v_pool, st, units)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        O.attention_rows(sc.cache, sc.k_pool, sc.v_pool, st, units)
    dt = time.perf_counter() - t0
    value = fl * args.steps / dt / 1e12
    sample = f"{len(units)} (request,row,head) units per step ({fl:.3g} flop) of workload {sc.name}"
    print(json.dumps({
        "impl": "reference", "metric": "chunk_attention_tflops", "value": value, "unit": "TFLOP/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": sc.name, "note": "CPU oracle on a bounded sample of the batch per step"},
        "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": O.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--workload", default="mixed_13b", choices=sorted(W.WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--q-group", type=int, default=1,
                    help="query heads per K/V head (spec_verify and mixed_13b only; the paper's models have 1)")
    ap.add_argument("--out16", action="store_true",
                    help="device-resident timing through hat_chunk_attention_out16 (output in the cache's 16-bit type); "
                         "the e2e leg keeps the fp32 host entry point")
    ap.add_argument("--graph", action="store_true",
                    help="capture the launch set of one step in a CUDA graph and time its replays (for the launch-bound "
                         "workloads); the per-kernel figures then come from a separate pass of ordinary launches")
    ap.add_argument("--tree", action="store_true",
                    help="token trees instead of linear drafts on the short chunks (spec_verify and mixed_13b only)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--all-configs", dest="all_configs", action="store_true", default=None,
                    help="after the main measurement, time the other named workloads briefly (default: on for the default "
                         "workload on one GPU)")
    ap.add_argument("--no-all-configs", dest="all_configs", action="store_false")
    ap.add_argument("--layer-front", dest="layer_front", action="store_true", default=None,
                    help="also time the projection kernel in front of the attention step (default: with --all-configs)")
    ap.add_argument("--cpu-budget", type=float, default=12.0, help="seconds of oracle work for cpu_baseline")
    args = ap.parse_args()
    if args.all_configs is None:
        args.all_configs = args.workload == "mixed_13b" and args.gpus == 1 and args.q_group == 1 and not args.tree
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        if args.steps is None:
            args.steps = 5
        if args.warmup is None:
            args.warmup = 1
        run_reference(args, rank)
        return
    if args.steps is None:
        args.steps = 1000 if args.workload in ("mixed_13b", "ragged_prefill", "spec_verify") else 200
    if args.warmup is None:
        args.warmup = 20
    args.warmup = max(args.warmup, 3)

    import torch
    import torch.distributed as dist
    from paper_2503_18989_b200 import binding as B
    from paper_2503_18989_b200 import build as hat_build
    from paper_2503_18989_b200 import runner

    if rank == 0:
        hat_build.build()
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)
        dist.barrier()

    def barrier():
        if world > 1:
            dist.barrier()

    peaks, peak_kind = load_peaks()

    # ---- inputs: one replica of the batch per rank (seeded; different values per rank)
    sc = make_workload(args, seed=replica_seed(args.workload, rank))
    cache = runner.DeviceCache(sc.cache, sc.k_pool, sc.v_pool, device)
    steps = [runner.DeviceStep(cache, st) for st in sc.steps]
    works = [step_work(sc.cache, st) for st in sc.steps]
    total = {k: sum(w[k] for w in works) for k in works[0]}
    kv_resident = 2 * sc.k_pool.nbytes
    flush_l2 = total["kv_bytes"] / len(sc.steps) < 2 * L2_BYTES
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=device) if flush_l2 else None
    stream = torch.cuda.current_stream(device).cuda_stream

    def one_step():
        for ds in steps:
            if args.out16:
                ds.attend16(fused_append=True, stream=stream)
            else:
                ds.attend(fused_append=True, stream=stream)

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize(device)
    for ds in steps:
        if B.hat_last_device_status(ds.plan, stream) != B.HAT_OK:
            raise RuntimeError("device-side wait timed out during warm-up")

    sampler = ClockSampler(local_rank)
    sampler.start()
    time.sleep(0.3)

    # ---- timed region: exactly K steps, device events, per-kernel events recorded by the library
    K = args.steps
    run_step, launches_per_replay = one_step, 0
    if args.graph:
        gstream = torch.cuda.Stream(device=device)
        gstream.wait_stream(torch.cuda.current_stream(device))
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(gstream):
            n0 = B.hat_launch_count()
            with torch.cuda.graph(graph, stream=gstream):
                for ds in steps:
                    (ds.attend16 if args.out16 else ds.attend)(fused_append=True, stream=gstream.cuda_stream)
            launches_per_replay = B.hat_launch_count() - n0
        torch.cuda.current_stream(device).wait_stream(gstream)
        run_step = graph.replay
        for _ in range(3):
            run_step()
    else:
        for ds in steps:
            B.hat_plan_enable_timing(ds.plan, K)
    launches0 = B.hat_launch_count()
    barrier(); torch.cuda.synchronize(device)
    t_wall0 = time.time()
    if not flush_l2:
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(K):
            run_step()
        e1.record()
        torch.cuda.synchronize(device)
        elapsed_ms = e0.elapsed_time(e1)
    else:
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        for a, b in evs:
            flush_buf.zero_()                 # evict the KV working set from L2 (not timed)
            a.record(); run_step(); b.record()
        torch.cuda.synchronize(device)
        elapsed_ms = sum(a.elapsed_time(b) for a, b in evs)
    t_wall1 = time.time()
    barrier()
    launches = B.hat_launch_count() - launches0 + launches_per_replay * K
    Kk = K
    if args.graph:
        # per-kernel durations cannot be read from events inside a graph: one more pass of ordinary launches
        Kk = min(K, 50)
        for ds in steps:
            B.hat_plan_enable_timing(ds.plan, Kk)
        for _ in range(Kk):
            if flush_l2:
                flush_buf.zero_()
            one_step()
        torch.cuda.synchronize(device)
    kernel_ms = np.zeros(B.HAT_TIMING_SLOTS)
    kernel_calls = np.zeros(B.HAT_TIMING_SLOTS)
    for ds in steps:
        ms = B.hat_plan_read_timing(ds.plan, Kk)
        kernel_ms += ms.sum(axis=0)
        kernel_calls += (ms > 0).sum(axis=0)
    clocks = sampler.summary(t_wall0, t_wall1)

    # ---- end to end through the host-buffer entry point: H2D of q/k_new/v_new and D2H of out/lse per step
    Ke = max(1, min(K, 100))
    # Two steps in flight: step i+1's host-to-device copies run on a second stream (with its own staging and result
    # buffers) while step i computes and copies its results back; the library itself keeps the calls of one plan in order.
    n_fly = 2
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a).view(np.int16)).pin_memory()
    host_in = [(pin(st.q), pin(st.k_new), pin(st.v_new)) for st in sc.steps]
    host = []
    for f in range(n_fly):
        bufs = []
        for ds, st in zip(steps, sc.steps):
            T, H, d = st.total_rows, int(st.q.shape[1]), sc.cache.head_dim
            nb = B.hat_plan_staging_bytes(ds.plan)
            bufs.append((torch.empty((T, H, d), dtype=torch.float32).pin_memory(),
                         torch.empty((T, H), dtype=torch.float32).pin_memory(),
                         torch.empty(max(nb, 256), dtype=torch.uint8, device=device), nb))
        host.append(bufs)
    fly_streams = [torch.cuda.Stream(device=device) for _ in range(n_fly)]

    def one_step_host(i):
        f = i % n_fly
        s_f = fly_streams[f].cuda_stream
        for ds, (q, k, v), (o, l, stg, nb) in zip(steps, host_in, host[f]):
            B.hat_chunk_attention_host(cache.desc, ds.plan, q, k, v, o, l, 0.0, stg, nb, ds.workspace,
                                       ds.workspace_bytes, s_f)
    for i in range(4):
        one_step_host(i)
    barrier(); torch.cuda.synchronize(device)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    main = torch.cuda.current_stream(device)
    e0.record(main)
    for fs in fly_streams:
        fs.wait_event(e0)
    for i in range(Ke):
        one_step_host(i)
    for fs in fly_streams:
        main.wait_stream(fs)
    e1.record(main)
    torch.cuda.synchronize(device)
    e2e_ms = e0.elapsed_time(e1)
    barrier()
    sampler.stop()
    h2d = sum(st.q.nbytes + st.k_new.nbytes + st.v_new.nbytes for st in sc.steps)
    d2h = sum(st.total_rows * int(st.q.shape[1]) * (sc.cache.head_dim + 1) * 4 for st in sc.steps)

    # ---- max over ranks
    elapsed_ms, e2e_ms = max_over_ranks([elapsed_ms, e2e_ms], world, device)

    if rank == 0:
        ms_per_step = elapsed_ms / K
        value = whole_job_value(total["flops"], world, ms_per_step)
        e2e_value = whole_job_value(total["flops"], world, e2e_ms / Ke)

        # per-kernel achieved throughput against its roofline
        timed_seconds = elapsed_ms * 1e-3
        tensor_peak, tensor_source = pick_tensor_peak(peaks, peak_kind, timed_seconds, clocks.get("reasons"))
        kernels = kernel_table(total, works, len(sc.steps), kernel_ms, kernel_calls, peaks, tensor_peak)
        dominant = max(kernels, key=lambda n: kernels[n]["share"])
        roof = {k: kernels[dominant][k] for k in ("bound", "achieved", "peak", "unit", "frac")}
        for k in ("frac_burst", "frac_sustained", "frac_nominal"):
            if k in kernels[dominant]:
                roof[k] = kernels[dominant][k]
        traffic = lookup_traffic(dominant, sc.name)
        alg_bytes = kernels[dominant].get("algorithmic_bytes")
        if alg_bytes is None and kernels[dominant]["bound"] == "hbm":
            alg_bytes = int(kernels[dominant]["achieved"] * 1e9 * kernels[dominant]["ms_per_launch"] * 1e-3)
        roof.update({"kernel": dominant, "traffic": traffic, "algorithmic_bytes": alg_bytes,
                     "traffic_over_algorithmic": (traffic / alg_bytes) if (traffic and alg_bytes) else None,
                     "peak_source": tensor_source if roof["bound"] == "tensor" else f"{peak_kind} HBM copy",
                     "timed_seconds": timed_seconds,
                     "ms_per_launch_x_sm_mhz": (kernels[dominant]["ms_per_launch"] * clocks["sm_mhz"])
                     if clocks.get("sm_mhz") else None})

        line = {
            "metric": "chunk_attention_tflops", "value": value, "unit": "TFLOP/s", "n_gpus": world,
            "steps": K, "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": sc.cache.dtype + " in, f32 accumulate",
            "data": "synthetic",
            "config": {"workload": sc.name, "requests": int(sc.steps[-1].num_requests), "rows": total["rows"],
                       "heads": int(sc.steps[-1].q.shape[1]), "kv_heads": sc.cache.num_heads,
                       "launch": "cuda graph replay" if args.graph else "stream launches",
                       "token_trees": bool(args.tree), "out": "16-bit" if args.out16 else "f32", "head_dim": sc.cache.head_dim, "page_size": 16,
                       "calls_per_step": len(sc.steps), "kv_resident_bytes": int(kv_resident),
                       "l2": "flushed between steps" if flush_l2 else "KV working set larger than L2",
                       "parallelism": f"replicas x{world}" if world > 1 else "1 gpu"},
            "e2e": {"value": e2e_value, "unit": "TFLOP/s", "h2d_bytes_per_step": int(h2d),
                    "d2h_bytes_per_step": int(d2h), "steps": Ke, "ms_per_step": e2e_ms / Ke,
                    "in_flight": "2 steps on 2 streams (copies of one step overlap the other's compute and copies)"},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": roof,
            "kernels": kernels,
            "kv_gbs": world * total["kv_bytes"] / (ms_per_step * 1e-3) / 1e9,
            "step_roofline": step_bound(total, ms_per_step, peaks, tensor_peak),
            "plan": steps[-1].info,
        }
        # Close the paper's control loop on the measured delay (Sec. 3.2-3.3, 3.5): one observation of (batched token
        # size, delay of this attention step), then the chunk size and parallel-drafting steps the controller would
        # hand to a device with the paper's WiFi rates (7.5 MB/s up, 12.5 MB/s down, 20 ms per drafting step).
        try:
            ctrl = B.Ctrl(0.8, 64.0, 256, 1)
            B.hat_ctrl_observe(ctrl, float(total["rows"]), ms_per_step * 1e-3)
            B.hat_ctrl_device_observe(ctrl, 0, 0.020, 7.5e6, 12.5e6)
            a_bytes = float(sc.cache.num_heads * sc.cache.head_dim * 2)
            line["controller"] = {
                "mu_tokens": B.hat_ctrl_mu(ctrl), "g_seconds": B.hat_ctrl_predict(ctrl, B.hat_ctrl_mu(ctrl)),
                "chunk_size_eq3": B.hat_ctrl_chunk_size(ctrl, 0, a_bytes, 1, 16, 2048),
                "parallel_draft_steps_eq6": B.hat_ctrl_parallel_draft_steps(ctrl, 0, 4, a_bytes),
                "note": "g holds one observation of this attention step alone, not of a whole middle-submodel step"}
            ctrl.close()
        except Exception as exc:                     # the controller is a report item, never a reason to lose the line
            line["controller"] = {"error": str(exc)}
        if not args.no_cpu_baseline and world == 1:
            rate, cores, sample, _, _ = time_oracle(sc, args.cpu_budget)
            line["cpu_baseline"] = {"value": rate / 1e12, "unit": "TFLOP/s", "cores": cores, "kind": "oracle",
                                    "sample": sample}
        if (args.layer_front or (args.layer_front is None and args.all_configs)) and world == 1:
            try:
                line["layer_front"] = layer_front(sc, cache, steps[0], device, stream, peaks, peak_kind,
                                                  with_oracle=not args.no_cpu_baseline)
            except Exception as exc:
                line["layer_front"] = {"error": str(exc)}
        if args.all_configs and world == 1:
            # the other named workloads, briefly, so that all five are in this run's record (parity cases, not the
            # headline: the line's value and roofline stay those of config.workload)
            for ds in steps:
                ds.close()
            del steps, cache, flush_buf, host, host_in
            torch.cuda.empty_cache()
            line["all_configs"] = {}
            for name in W.WORKLOADS:
                if name == sc.name:
                    continue
                try:
                    line["all_configs"][name] = quick_config(name, device, stream, peaks, peak_kind,
                                                             with_oracle=not args.no_cpu_baseline)
                except Exception as exc:
                    line["all_configs"][name] = {"error": str(exc)}
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()

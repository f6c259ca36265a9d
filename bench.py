#!/usr/bin/env python
"""Benchmark of the PISA forward hot path (pyramid -> routing -> block-sparse attention).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg4] [--impl ours|reference]

One "step" is one pass of the whole path over one batch of synthetic input.  Prints ONE JSON line
(rank 0).  `value` is forward tokens/s with inputs resident in HBM; `e2e` is the same metric through
pisa_forward_host (pinned host tensors in, host tensors out, copies inside the timed region).
`--impl reference` times the CPU oracle, as it stands, on a bounded sample of the same workload.
Multi-GPU: the path shards over independent (batch, KV head) units with no exchange step, so every
rank runs its own replica of the workload (weak scaling) and no collective is on the data path.
"""
from __future__ import annotations

import argparse
import dataclasses
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import pisa_synth as S  # noqa: E402

METRIC = "pisa_fwd_tokens_per_s_128k_ctx"
UNIT = "tokens/s"



def dram_bytes_per_pair() -> dict:
    """dram__bytes_read.sum + dram__bytes_write.sum per selected (token, block) pair of the two tile
    kernels, read from the file that is written with the ncu captures (profiles/)."""
    try:
        d = json.load(open(os.path.join(ROOT, "profiles", "dram_bytes_per_pair.json")))
        n = float(d["pairs_per_launch"])
        return {k_: (v_["dram_bytes_read"] + v_["dram_bytes_write"]) / float(v_.get("pairs_per_launch", n))
                for k_, v_ in d.items() if isinstance(v_, dict)}
    except Exception:
        return {}


def get_workload(name: str) -> S.Workload:
    if name in S.WORKLOADS:
        return S.WORKLOADS[name]
    if name.startswith("cfg5_"):
        return S.sweep_workload(int(name.split("_")[1]))
    if name.startswith("custom:"):       # custom:B,N,Hq,Hkv,d,C,g,K  (bf16, i.i.d., for profiling captures)
        B, N, Hq, Hkv, d, C, g, K = (int(x) for x in name.split(":")[1].split(","))
        return S.Workload(name, B, N, Hq, Hkv, d, C, g, K, "bf16", 9, "iid")
    raise SystemExit(f"unknown workload {name}")


def describe(w: S.Workload) -> str:
    return (f"{w.name}: B={w.B} Hq={w.Hq} Hkv={w.Hkv} d={w.d} N={w.N} causal C={w.C} g={w.g} K={w.K} "
            f"{w.dtype} {w.structure} seed={w.seed}")


# ------------------------------------------------------------------ algorithmic work counts

def work_counts(w: S.Workload) -> dict:
    """Integer bookkeeping of what one forward pass must touch (depends on shapes only, not data):
    scored (token, node) pairs per level and selected (token, block) pairs."""
    M = [w.N, -(-w.N // w.C)]
    while M[-1] > 1:
        M.append(-(-M[-1] // w.g))
    L = len(M) - 1
    inter_pairs = 0      # (token, candidate) pairs scored from child summaries, summed over levels >= 2
    leaf_pairs = 0       # (token, leaf) pairs scored from raw keys
    sel_pairs = 0        # (token, selected leaf) pairs
    forced_pairs = 0     # of those, the forced leaves (first / previous / current), served by the local-window kernel
    for c in range(M[1]):
        toks = min(w.C, w.N - c * w.C)
        n_kept = 1
        kept_has_anc = True
        for l in range(L, 0, -1):
            span = w.g ** (l - 1)
            anc = c // span
            if l == L:
                nV = 1
            else:
                # children of the kept nodes; those of the current ancestor beyond anc are dropped
                anc_up = c // (w.g ** l)
                full = (n_kept - 1) * w.g
                nV = full + (anc - anc_up * w.g + 1)
            forced = len({0, anc, (c - 1) // span if c >= 1 else 0})
            if nV > w.K:
                if l >= 2:
                    inter_pairs += toks * (nV - forced)
                else:
                    leaf_pairs += toks * (nV - forced)
                n_kept = w.K
            else:
                n_kept = nV
        sel_pairs += toks * n_kept
        forced_pairs += toks * min(3, c + 1)
    units = w.B * w.Hkv
    G = w.Hq // w.Hkv
    es = 2 if w.dtype == "bf16" else 4
    return {
        "inter_flops": 2.0 * inter_pairs * w.g * G * w.d * units,
        "leaf_flops": 2.0 * leaf_pairs * w.C * G * w.d * units,
        "attn_flops": 4.0 * sel_pairs * w.C * G * w.d * units,
        "pyramid_bytes": float(w.B * w.N * w.Hkv * w.d * es + w.B * w.Hkv * sum(M[1:]) * w.d * es),
        "hbm_min_bytes": float(w.B * w.N * ((2 * w.Hq + 2 * w.Hkv) * w.d * es + w.Hq * 4 + w.Hkv * w.K * 4)),
        "sel_pairs": sel_pairs * units, "leaf_pairs": leaf_pairs * units, "inter_pairs": inter_pairs * units,
        "forced_pairs": forced_pairs * units, "forced_flops": 4.0 * forced_pairs * w.C * G * w.d * units,
    }


# ------------------------------------------------------------------ clocks

class ClockSampler:
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_id: str):
        self.lines = []
        self.proc = None
        self.gpu_id = gpu_id
        self.first = 0              # index of the first sample that belongs to the timed region

    def mark(self):
        """The timed region starts now: samples taken before this call are dropped."""
        self.first = len(self.lines)

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", self.gpu_id, f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "25"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        n_end = len(self.lines)       # samples that arrived while the timed region ran
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines[self.first:max(n_end, self.first + 1)]:
            parts = [x.strip() for x in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# ------------------------------------------------------------------ CPU oracle legs

def oracle_sample_rate(w: S.Workload, tensors: dict, n_queries: int, seed: int = 0, threads: int = 0):
    """Times the compiled oracle (oracle/pisa_oracle_c.c, as it stands) on one (batch, KV head) unit: its
    pyramid in full plus `n_queries` sampled query positions of it (routing + attention of the group's
    heads), on `threads` host threads (0 = all the box has).  Returns the whole-workload tokens/s this
    extrapolates to, the seconds spent, the threads used and a description of the sample."""
    from oracle import pisa_oracle_c as OC
    rng = np.random.default_rng(seed)
    h = int(rng.integers(0, w.Hkv))
    ps = np.sort(rng.integers(0, w.N, size=n_queries))
    prob = OC.CProblem(tensors["q"], tensors["k"], tensors["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype, threads=threads)
    t0 = time.perf_counter()
    prob.unit(0, h)                                   # widens the unit's keys and pools its pyramid
    t1 = time.perf_counter()
    tri = np.stack([np.zeros_like(ps), np.full_like(ps, h), ps], axis=1)
    idx, _ = prob.route_all(tri)
    prob.attend_all(tri, idx)
    t2 = time.perf_counter()
    per_unit = (t1 - t0) + (t2 - t1) / n_queries * w.N
    total = per_unit * w.B * w.Hkv
    return (w.B * w.N) / total, (t2 - t0), prob.threads, (
        f"compiled oracle, {prob.threads} thread(s): pyramid of 1 of {w.B * w.Hkv} (batch, KV head) units in full + "
        f"{n_queries} uniformly sampled query positions of it (route + attention of its {w.Hq // w.Hkv} heads), "
        f"scaled by N/{n_queries} and by the unit count")


def cpu_baseline_leg(w: S.Workload, tensors: dict, n_queries: int) -> dict:
    """The oracle on the machine's host cores: all cores on `n_queries` sampled positions, one core on a quarter."""
    val, secs, cores, sample = oracle_sample_rate(w, tensors, n_queries)
    val1, secs1, _, _ = oracle_sample_rate(w, tensors, max(64, n_queries // 4), threads=1)
    return {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample, "seconds": secs,
            "host_cores": os.cpu_count(), "value_1_thread": val1, "seconds_1_thread": secs1}


def parity_of_timed_buffers(w: S.Workload, tensors: dict, idx, out, lse, per_unit: int = 64) -> dict:
    """Checks the buffers a timed run left behind against the oracle on sampled rows (at least 256 at the
    headline shape): index sets (a differing row is excused only if the oracle's cut margin of that row is
    inside the 1e-4 tie band), then outputs and denominators of every sampled row against the oracle's
    attention on the sets the GPU selected.  idx / out / lse: torch tensors (device or host)."""
    import torch
    from oracle import pisa_oracle_c as OC
    tri = S.sample_queries(w, per_unit)
    prob = OC.CProblem(tensors["q"], tensors["k"], tensors["v"], C=w.C, g=w.g, K=w.K, dtype=w.dtype)
    ref_idx, margin = prob.route_all(tri)
    t = torch.from_numpy(tri).to(idx.device)
    got = idx[t[:, 0], t[:, 1], t[:, 2]].cpu().numpy()
    differ = np.any(got != ref_idx, axis=1)
    out_ref, lse_ref = prob.attend_all(tri, got)
    G = w.Hq // w.Hkv
    heads = t[:, 1:2] * G + torch.arange(G, device=idx.device)[None, :]
    o = out[t[:, 0:1], t[:, 2:3], heads].to(torch.float64).cpu().numpy()
    l = lse[t[:, 0:1], heads, t[:, 2:3]].to(torch.float64).cpu().numpy()
    err = np.abs(o - out_ref)
    return {"rows": int(len(tri)), "rows_differ": int(differ.sum()), "rows_differ_outside_tie_band": int((differ & (margin > 1e-4)).sum()),
            "rows_in_tie_band": int((margin <= 1e-4).sum()), "out_max_abs": float(err.max()), "out_mean_abs": float(err.mean()),
            "lse_max_abs": float(np.abs(l - lse_ref).max()),
            "ok": bool((differ & (margin > 1e-4)).sum() == 0 and err.max() <= (2e-2 if w.dtype == "bf16" else 1e-4)
                       and err.mean() <= (2e-3 if w.dtype == "bf16" else 1e-4))}


def run_reference(args):
    rank = rank_env()[0]
    if rank != 0:             # under torchrun only rank 0 runs the CPU reference
        return
    w = get_workload(args.workload)
    tensors = S.make_inputs(w)
    nq = args.ref_queries
    for _ in range(args.warmup):
        oracle_sample_rate(w, tensors, max(4, nq // 8), seed=99)
    t0 = time.perf_counter()
    rates = []
    cores = 1
    for s in range(args.steps):
        r, _, cores, sample = oracle_sample_rate(w, tensors, nq, seed=s)
        rates.append(r)
    wall = time.perf_counter() - t0
    value = float(len(rates) / sum(1.0 / r for r in rates))
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": wall / max(1, args.steps) * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": describe(w)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


# ------------------------------------------------------------------ multi-rank plumbing

def rank_env():
    return (int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")),
            int(os.environ.get("LOCAL_RANK", "0")))


def replica_workload(w: S.Workload, rank: int) -> S.Workload:
    """The path shards over independent (batch, KV head) units without any exchange step, so rank r
    simply owns its own replica of the workload (same shape, its own seed): weak scaling."""
    return dataclasses.replace(w, seed=w.seed + 1000 * rank)


def max_over_ranks(values, world: int, device=None):
    """Element-wise max of a list of floats over all ranks (identity for one rank)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def job_tokens_per_s(w: S.Workload, world: int, steps: int, ms: float) -> float:
    """Whole-job throughput: every rank processed B*N tokens per step in `ms` (max over ranks)."""
    return world * w.B * w.N * steps / (ms * 1e-3)


# ------------------------------------------------------------------ our arm

def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2609_31093_b200 as P
    from paper_2609_31093_b200 import binding as PB

    rank, world, local = rank_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the path has no CPU fallback")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    w0 = get_workload(args.workload)
    w = replica_workload(w0, rank)
    impl = {"auto": PB.IMPL_AUTO, "simt": PB.IMPL_SIMT, "tensor": PB.IMPL_TENSOR}[args.path]
    p = P.Params.from_workload(w, impl=impl)
    tensors = S.make_inputs(w)
    tdt = p.torch_dtype

    def host(a):
        t = torch.from_numpy(a.view(np.int16)).view(torch.bfloat16) if w.dtype == "bf16" else torch.from_numpy(a)
        return t.pin_memory()

    qh, kh, vh = host(tensors["q"]), host(tensors["k"]), host(tensors["v"])
    q, k, v = qh.cuda(non_blocking=True), kh.cuda(non_blocking=True), vh.cuda(non_blocking=True)
    pyramid = PB.alloc_pyramid(p)
    idx = torch.empty((w.B, w.Hkv, w.N, w.K), dtype=torch.int32, device="cuda")
    out = torch.empty_like(q)
    lse = torch.empty((w.B, w.Hq, w.N), dtype=torch.float32, device="cuda")
    ws = PB.alloc_workspace(p, PB.OP_FORWARD)
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()

    P.set_forward_chunks(args.forward_chunks)

    def step():
        P.pisa_forward(p, q, k, v, pyramid, idx, out, lse, ws)

    props = torch.cuda.get_device_properties(local)
    gpu_id = str(local)
    if hasattr(props, "uuid"):
        u = str(props.uuid)
        gpu_id = u if u.startswith("GPU-") else "GPU-" + u
    sampler = ClockSampler(gpu_id)
    sampler.start()                  # nvidia-smi takes a moment to come up: it runs through the warm-up
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    st = P.read_status(ws)
    if st != 0:
        raise SystemExit(f"device status {st} after warm-up")

    P.set_stage_timing(True)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    stage = np.zeros(3)
    kernels = {}
    launches_of = {}
    barrier()
    torch.cuda.synchronize()
    sampler.mark()
    l0 = P.launch_count()
    ev0.record()
    for _ in range(args.steps):
        step()
        stage += np.asarray(P.get_stage_ms())       # waits for this step's last event
        for name, t_ms in P.get_kernel_brackets():
            kernels[name] = kernels.get(name, 0.0) + t_ms
            launches_of[name] = launches_of.get(name, 0) + 1
    ev1.record()
    torch.cuda.synchronize()
    launches = P.launch_count() - l0
    clocks = sampler.stop()
    barrier()
    ms = ev0.elapsed_time(ev1)
    stage /= args.steps
    # In the timed region a large forward runs as chunks on two streams, so a bracket there is the span
    # of a launch that shares the GPU with the other stream's kernels.  Each kernel alone: a few more
    # steps, untimed, with the chunking off (these are the times the serialised ncu launch list shows).
    spans = {k_: v_ / args.steps for k_, v_ in kernels.items()}
    launches_of = {k_: v_ // args.steps for k_, v_ in launches_of.items()}
    P.set_forward_chunks(1)
    kernels = {}
    n_serial = 2
    for _ in range(n_serial):
        step()
        P.get_stage_ms()
        for name, t_ms in P.get_kernel_ms().items():
            kernels[name] = kernels.get(name, 0.0) + t_ms / n_serial
    P.set_forward_chunks(args.forward_chunks)
    P.set_stage_timing(False)

    # end to end through the host-buffer entry point
    arena = PB.alloc_workspace(p, PB.OP_FORWARD_HOST)
    out_h = torch.empty(q.shape, dtype=tdt).pin_memory()
    lse_h = torch.empty(lse.shape, dtype=torch.float32).pin_memory()
    idx_h = torch.empty(idx.shape, dtype=torch.int32).pin_memory()
    e2e_steps = max(0, min(args.steps, args.e2e_steps))
    e2e_ms = float("nan")
    if e2e_steps > 0:
        for _ in range(2):
            P.pisa_forward_host(p, qh, kh, vh, out_h, lse_h, None, arena)
        barrier()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(e2e_steps):
            P.pisa_forward_host(p, qh, kh, vh, out_h, lse_h, None, arena)
        e1.record()
        torch.cuda.synchronize()
        barrier()
        e2e_ms = e0.elapsed_time(e1)

    ms, e2e_ms = max_over_ranks([ms, e2e_ms], world, device="cuda")
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    value = job_tokens_per_s(w, world, args.steps, ms)
    e2e_value = job_tokens_per_s(w, world, e2e_steps, e2e_ms) if e2e_steps > 0 else None
    wc = work_counts(w)
    peaks = {}
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        pass
    hbm_peak = peaks.get("hbm_gbs", 6650.0)
    tens_peak = peaks.get("bf16_tflops_sustained", 1400.0)
    peak_src = "measured" if peaks else "fallback"
    es = 2 if w.dtype == "bf16" else 4
    # Roofline entry for the dominant kernel, timed live with CUDA events on the launching stream.
    # Algorithmic work per launch: leaf scoring and attention are dense contractions (tensor bound,
    # 2*C*G*d flops per scored (token, leaf) pair, 4*C*G*d per selected pair), the intermediate levels
    # too (2*g*G*d per scored (token, node) pair); the pyramid is one streaming pass over k (HBM bound).
    # with the local-window kernel in the launch list the list-driven attention kernel only sees the routed pairs
    local = "local_window" in kernels
    routed_flops = wc["attn_flops"] - (wc["forced_flops"] if local else 0.0)
    routed_pairs = wc["sel_pairs"] - (wc["forced_pairs"] if local else 0)
    algo = {
        "leaf_lse_tiles": ("tensor", wc["leaf_flops"]), "attention_tiles": ("tensor", routed_flops),
        "local_window": ("tensor", wc["forced_flops"]),
        "route_stage1": ("tensor", wc["inter_flops"]), "route_simt": ("tensor", wc["leaf_flops"] + wc["inter_flops"]),
        "bsa_simt": ("tensor", wc["attn_flops"]), "pyramid": ("hbm", wc["pyramid_bytes"]),
    }
    cand = {k_: v_ for k_, v_ in kernels.items() if k_ in algo}
    dom = max(cand, key=cand.get) if cand else "pyramid"          # by its time alone
    bound, work = algo[dom]
    t_alone = cand.get(dom, stage[0]) * 1e-3
    t_dom = spans.get(dom, cand.get(dom, stage[0])) * 1e-3         # summed launch spans inside the timed region
    if bound == "hbm":
        roof = {"kernel": dom, "bound": "hbm", "achieved": work / t_dom / 1e9, "peak": hbm_peak, "unit": "GB/s"}
    else:
        roof = {"kernel": dom, "bound": "tensor", "achieved": work / t_dom / 1e12, "peak": tens_peak,
                "unit": "TFLOP/s"}
    # `achieved` / `frac`: the kernel ALONE on the GPU (the whole problem as one launch, chunking off), which
    # is what a per-kernel roofline means; the launch spans inside the timed region, where a launch shares
    # the SMs with the other stream's kernels, are kept beside them as in_step_*
    roof["in_step_achieved"] = roof["achieved"]
    roof["in_step_frac"] = roof["achieved"] / roof["peak"]
    roof["achieved"] = work / t_alone / (1e9 if bound == "hbm" else 1e12)
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["peak_source"] = peak_src + (" (sustained bf16, kernel timed inside a long step)" if bound == "tensor" else "")
    n_launch = max(1, launches_of.get(dom, 1))                    # one launch per chunk
    roof["launch_ms"] = t_dom * 1e3 / n_launch                    # average launch; achieved = (work / n) / this
    roof["launches_per_step"] = n_launch
    roof["alone_ms"] = t_alone * 1e3                               # the whole problem as one launch, GPU to itself
    roof["frac_of_burst_peak"] = (work / t_alone / 1e12 / peaks.get("bf16_tflops", 1590.0)) if bound == "tensor" else None
    # DRAM bytes per launch from the ncu capture of a smaller case of the same kernel (summary under
    # profiles/), scaled by the (token, block) pairs a launch processes: traffic grows with the pairs
    per_pair = dram_bytes_per_pair().get(dom)
    pairs = {"leaf_lse_tiles": wc["sel_pairs"], "attention_tiles": routed_pairs}.get(dom)
    roof["traffic"] = (per_pair * pairs / n_launch) if (per_pair and pairs and w.dtype == "bf16") else None
    # The two tile kernels are limited by what L2 can gather and reduce, not by the tensor pipe: report
    # that stream too (per selected pair: G*d*2 bytes of query rows L2->SM, and in the attention
    # kernel G*d*4 bytes of fp32 reductions SM->L2).  Context for `frac`, not a substitute for it.
    if dom in ("leaf_lse_tiles", "attention_tiles") and w.dtype == "bf16":
        per_pair_l2 = w.G * w.d * 2 + (w.G * w.d * 4 if dom == "attention_tiles" else 0)
        l2_pairs = routed_pairs if dom == "attention_tiles" else wc["sel_pairs"]
        roof["l2_stream_bytes"] = per_pair_l2 * l2_pairs / n_launch
        roof["l2_stream_tbs"] = per_pair_l2 * l2_pairs / t_alone / 1e12
    roofs = {}
    for k_, t_ in cand.items():
        b_, w_ = algo[k_]
        roofs[k_] = {"ms": t_, ("gbs" if b_ == "hbm" else "tflops"): w_ / (t_ * 1e-3) / (1e9 if b_ == "hbm" else 1e12),
                     "frac": w_ / (t_ * 1e-3) / ((hbm_peak * 1e9) if b_ == "hbm" else (tens_peak * 1e12))}
        if k_ == "route_stage1":
            # gathered per-token products on warp-level MMAs: bound by instruction issue (ncu: about 70 % of the
            # issue slots busy), not by the tensor pipe -- a fraction of the tensor peak would say nothing
            roofs[k_]["bound"] = "instruction issue"
            del roofs[k_]["frac"]
    # stage times from the kernels-alone pass (in the timed region the stages of different chunks overlap)
    t_pyr = kernels.get("pyramid", stage[0])
    t_route = sum(kernels.get(n_, 0.0) for n_ in ("route_stage1", "invert_by_parent", "leaf_lse_tiles", "final_topk",
                                                   "route_simt")) or stage[1]
    t_attn = sum(kernels.get(n_, 0.0) for n_ in ("invert_by_leaf", "accumulator_memset", "local_window", "attention_tiles",
                                                  "convert_out", "bsa_simt", "row_lse")) or stage[2]
    stages = {
        "pyramid_us": t_pyr * 1e3, "route_us": t_route * 1e3, "attn_us": t_attn * 1e3,
        "pyramid_gbs": wc["pyramid_bytes"] / (t_pyr * 1e-3) / 1e9,
        "route_tflops": (wc["leaf_flops"] + wc["inter_flops"]) / (t_route * 1e-3) / 1e12,
        "attn_tflops": wc["attn_flops"] / (t_attn * 1e-3) / 1e12,
        "whole_step_hbm_min_gbs": wc["hbm_min_bytes"] / (ms / args.steps * 1e-3) / 1e9,
    }
    cpu = None
    parity = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline_leg(w, tensors, args.ref_queries)
    if world == 1 and not args.no_parity:
        # the buffers the timed region and the end-to-end region left behind, against the oracle
        parity = {"device_buffers": parity_of_timed_buffers(w, tensors, idx, out, lse)}
        if e2e_steps > 0:
            P.pisa_forward_host(p, qh, kh, vh, out_h, lse_h, idx_h, arena)
            parity["host_buffers"] = parity_of_timed_buffers(w, tensors, idx_h, out_h, lse_h)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": w.dtype, "data": "synthetic",
        "config": {"workload": describe(w0), "path": args.path,
                   "l2": f"inputs larger than L2 (q {q.numel() * es / 1e6:.0f} MB, k+v {2 * k.numel() * es / 1e6:.0f} MB)",
                   "replicas": world},
        "stages": stages, "kernels_ms": kernels, "kernels_ms_spans_in_timed_region": spans, "kernel_rooflines": roofs, "roofline": roof, "cpu_baseline": cpu, "parity": parity,
        "e2e": {"value": e2e_value, "unit": UNIT, "steps": e2e_steps,
                "h2d_bytes_per_step": int((q.numel() + 2 * k.numel()) * es),
                "d2h_bytes_per_step": int(out.numel() * es + lse.numel() * 4)},
        "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def run_sweep(args):
    """Routing latency vs N (the scaling-sweep workload) next to the flat O(N^2/C) selector built in the same
    library, plus the paper's own benchmark shape; one JSON line per (workload, N).  Not the bench line."""
    import torch

    import paper_2609_31093_b200 as P
    from paper_2609_31093_b200 import binding as PB

    torch.cuda.set_device(0)
    rows = []
    plans = [("cfg5", [8192, 32768, 131072, 524288], lambda n: S.sweep_workload(n)),
             ("paper_shape", [4096, 8192, 16384, 32768, 65536, 131072, 262144],
              lambda n: S.Workload(f"paper_{n}", 1, n, 32, 2, 64, 64, 2, 8, "bf16", 5, "iid"))]
    for tag, ns, mk in plans:
        for n in ns:
            w = mk(n)
            t = S.make_inputs(w)
            p = P.Params.from_workload(w)
            dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()
            q, k, v = dev(t["q"]), dev(t["k"]), dev(t["v"])
            pyramid = PB.alloc_pyramid(p)
            idx = torch.empty((w.B, w.Hkv, w.N, w.K), dtype=torch.int32, device="cuda")
            out = torch.empty_like(q)
            lse = torch.empty((w.B, w.Hq, w.N), dtype=torch.float32, device="cuda")
            ws = PB.alloc_workspace(p, PB.OP_FORWARD)

            def timed(fn, reps):
                for _ in range(2):
                    fn()
                torch.cuda.synchronize()
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                for _ in range(reps):
                    fn()
                e1.record()
                torch.cuda.synchronize()
                return e0.elapsed_time(e1) / reps

            reps = 5 if n <= 131072 else 2
            t_pyr = timed(lambda: P.pisa_build_pyramid(p, k, pyramid), reps)
            t_route = timed(lambda: P.pisa_route(p, q, k, pyramid, idx, None, ws), reps)
            t_flat = timed(lambda: P.pisa_flat_select(p, q, pyramid, idx, ws), 1 if n > 131072 else reps)
            t_fwd = timed(lambda: P.pisa_forward(p, q, k, v, pyramid, idx, out, lse, ws), reps)
            st = P.read_status(ws)
            row = {"sweep": tag, "workload": describe(w), "N": n, "pyramid_ms": t_pyr, "route_ms": t_route,
                   "selection_ms": t_pyr + t_route, "flat_select_ms": t_flat, "flat_selection_ms": t_pyr + t_flat,
                   "forward_ms": t_fwd, "forward_tokens_per_s": w.B * n / (t_fwd * 1e-3), "status": st,
                   "route_us_per_token": t_route * 1e3 / n}
            rows.append(row)
            print(json.dumps(row), flush=True)
            del q, k, v, pyramid, idx, out, lse, ws
            torch.cuda.empty_cache()
    return rows


def decode_bytes_per_step(w, pos):
    """Algorithmic bytes one decoding step must read for a late token (per the method, Sec. 3.3
    "Decoding"): child summaries of the scored candidates at every pruned intermediate level, the raw
    keys of the scored leaf candidates, keys and values of the selected blocks."""
    es, c = 2, pos // w.C
    M = [w.N, -(-w.N // w.C)]
    while M[-1] > 1:
        M.append(-(-M[-1] // w.g))
    L = len(M) - 1
    per_head = 0
    n = 1
    for l in range(L, 1, -1):
        anc = c // (w.g ** (l - 1))
        nV = min(n, anc + 1)
        if nV > w.K:
            per_head += nV * w.g * w.d * es
            nV = w.K
        n = nV * w.g
    nV1 = min(n, c + 1)
    if nV1 > w.K:
        per_head += (nV1 - 3) * w.C * w.d * es
    per_head += min(nV1, w.K) * w.C * w.d * es * 2
    return per_head * w.B * w.Hkv


def run_decode(args):
    """Decoding latency vs context length: one pisa_decode_step launch per token over a cache whose
    pyramid was built by the prefill kernels.  One JSON line per (shape, N).  Not the bench line."""
    import torch

    import paper_2609_31093_b200 as P
    from paper_2609_31093_b200 import binding as PB

    torch.cuda.set_device(0)
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        peaks = {}
    hbm_peak = peaks.get("hbm_gbs", 6650.0)
    shapes = [("cfg4_shape", dict(B=1, Hq=32, Hkv=8, d=128, C=128, g=2, K=32)),
              ("cfg5_shape", dict(B=1, Hq=16, Hkv=4, d=128, C=64, g=2, K=16)),
              ("paper_shape", dict(B=1, Hq=32, Hkv=2, d=64, C=64, g=2, K=8)),
              ("cfg4_shape_b8", dict(B=8, Hq=32, Hkv=8, d=128, C=128, g=2, K=32))]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for tag, sh in shapes:
        for n in [8192, 32768, 131072, 524288]:
            if sh["B"] * n * sh["Hkv"] * sh["d"] * 2 * 2 > 40e9:
                continue
            w = S.Workload(f"{tag}_{n}", sh["B"], n, sh["Hq"], sh["Hkv"], sh["d"], sh["C"], sh["g"], sh["K"],
                           "bf16", 6, "iid")
            p = P.Params.from_workload(w)
            gen = torch.Generator(device="cuda").manual_seed(1000 + n)
            k = torch.randn((w.B, n, w.Hkv, w.d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
            v = torch.randn((w.B, n, w.Hkv, w.d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
            steps = 32
            qs = torch.randn((steps, w.B, w.Hq, w.d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
            pyramid = PB.alloc_pyramid(p)
            P.pisa_build_pyramid(p, k, pyramid)
            idx = torch.empty((w.B, w.Hkv, w.K), dtype=torch.int32, device="cuda")
            out = torch.empty((w.B, w.Hq, w.d), dtype=torch.bfloat16, device="cuda")
            lse = torch.empty((w.B, w.Hq), dtype=torch.float32, device="cuda")
            ws = PB.alloc_workspace(p, PB.OP_DECODE)
            pos0 = n - steps
            for i in range(3):
                P.pisa_decode_step(p, pos0 + i, qs[i], k, v, pyramid, idx, out, lse, ws)
            torch.cuda.synchronize()
            # cold: L2 flushed before every step
            cold = 0.0
            evs = []
            for i in range(steps):
                flush.fill_(i & 0xFF)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                P.pisa_decode_step(p, pos0 + i, qs[i], k, v, pyramid, idx, out, lse, ws)
                e1.record()
                evs.append((e0, e1))
            torch.cuda.synchronize()
            cold = sum(a.elapsed_time(b) for a, b in evs) / steps * 1e3
            # warm: steps back to back
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for i in range(steps):
                P.pisa_decode_step(p, pos0 + i, qs[i], k, v, pyramid, idx, out, lse, ws)
            e1.record()
            torch.cuda.synchronize()
            warm = e0.elapsed_time(e1) / steps * 1e3
            nbytes = decode_bytes_per_step(w, n - 1)
            row = {"decode": tag, "workload": describe(w), "N": n, "us_per_step_cold_l2": cold,
                   "us_per_step_back_to_back": warm, "algorithmic_bytes_per_step": nbytes,
                   "gbs_cold": nbytes / (cold * 1e-6) / 1e9, "hbm_peak_gbs": hbm_peak,
                   "frac_hbm_cold": nbytes / (cold * 1e-6) / 1e9 / hbm_peak, "status": P.read_status(ws),
                   "tokens_per_s_back_to_back": w.B / (warm * 1e-6)}
            print(json.dumps(row), flush=True)
            del k, v, qs, pyramid
            torch.cuda.empty_cache()


def selection_quality(idx_sparse, mass):
    """Recall@K and MassRatio (Sec. 5 "Block-selection quality") of selected block sets against the
    reference sets built from full-attention block masses.

    idx_sparse: int array [S, K] (-1 padded); mass: float array [S, M] = full-attention mass of every
    block for the same S queries (already averaged over the group's heads, zero for future blocks).
    The reference set of a query is its K blocks of largest mass (among blocks with non-zero mass when
    fewer than K exist).  Returns (recall [S], mass_ratio [S])."""
    idx_sparse = np.asarray(idx_sparse)
    mass = np.asarray(mass, dtype=np.float64)
    S_, K = idx_sparse.shape
    recall = np.empty(S_)
    ratio = np.empty(S_)
    for s in range(S_):
        live = int((mass[s] > 0).sum())
        k_ref = min(K, live)
        ref = np.argsort(-mass[s], kind="stable")[:k_ref]
        sel = idx_sparse[s][idx_sparse[s] >= 0]
        recall[s] = len(set(ref.tolist()) & set(sel.tolist())) / float(max(k_ref, 1))
        ratio[s] = mass[s][sel].sum() / max(mass[s][ref].sum(), 1e-300)
    return recall, ratio


def run_quality(args):
    """Selection quality of the score modes (LSE = PISA, mean = PISA-1, mean + variance/2 = PISA-2) and of
    the flat mean selector against full attention, on synthetic tensors with a drifting mean (the
    paper measures this on a trained model's queries and keys, which are not available here; the
    numbers say how the selectors differ on this synthetic structure, nothing about a model).
    One JSON line per selector.  Not the bench line."""
    import torch

    import paper_2609_31093_b200 as P
    from paper_2609_31093_b200 import binding as PB

    torch.cuda.set_device(0)
    w = S.Workload("quality_walk", 1, 16384, 8, 2, 128, 64, 2, 8, "bf16", 7, "walk")
    t = S.make_inputs(w)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()
    q, k = dev(t["q"]), dev(t["k"])
    rng = np.random.default_rng(11)
    pos = np.sort(rng.choice(np.arange(w.K * w.C, w.N), size=512, replace=False))
    # full-attention block masses of the sampled queries, averaged over the group's heads
    G, M1 = w.G, w.M1
    mass = np.zeros((w.Hkv, len(pos), M1))
    scale = 1.0 / np.sqrt(w.d)
    for h in range(w.Hkv):
        kf = k[0, :, h].float()                                            # [N, d]
        for j, p_ in enumerate(pos.tolist()):
            qf = q[0, p_, h * G:(h + 1) * G].float()                       # [G, d]
            z = (qf @ kf[:p_ + 1].T) * scale
            pr = torch.softmax(z.double(), dim=-1).mean(dim=0)              # [p+1]
            pad = torch.zeros(M1 * w.C, dtype=torch.float64, device="cuda")
            pad[:p_ + 1] = pr
            mass[h, j] = pad.view(M1, w.C).sum(dim=1).cpu().numpy()
    rows = []
    for name, mode, impl, flat in (("pisa_lse", "lse", PB.IMPL_AUTO, False), ("pisa1_mean", "mean", PB.IMPL_AUTO, False),
                                   ("pisa2_mean_var", "mean_var", PB.IMPL_AUTO, False), ("flat_mean", "lse", PB.IMPL_AUTO, True)):
        p = P.Params.from_workload(w, score_mode=mode, impl=impl)
        pyramid = PB.alloc_pyramid(p)
        idx = torch.empty((w.B, w.Hkv, w.N, w.K), dtype=torch.int32, device="cuda")
        ws = PB.alloc_workspace(p, PB.OP_FORWARD)
        P.pisa_build_pyramid(p, k, pyramid)
        run = (lambda: P.pisa_flat_select(p, q, pyramid, idx, ws)) if flat else \
              (lambda: P.pisa_route(p, q, k, pyramid, idx, None, ws))
        run()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        run()
        e1.record()
        torch.cuda.synchronize()
        select_ms = e0.elapsed_time(e1)
        sel = idx[0][:, torch.from_numpy(pos).cuda()].cpu().numpy()         # [Hkv, S, K]
        rec, rat = [], []
        for h in range(w.Hkv):
            r_, m_ = selection_quality(sel[h], mass[h])
            rec.append(r_)
            rat.append(m_)
        row = {"quality": name, "workload": describe(w), "queries": int(len(pos) * w.Hkv), "K": w.K,
               "recall_at_k": float(np.mean(rec)), "mass_ratio": float(np.mean(rat)), "select_ms": select_ms,
               "path": "flat SIMT" if flat else ("tcgen05 + mma.sync" if impl == PB.IMPL_AUTO else "SIMT fp32"),
               "status": P.read_status(ws)}
        rows.append(row)
        print(json.dumps(row), flush=True)
    return rows


def run_backward(args):
    """Backward of the block-sparse attention (frozen indices) at the requested workload: forward once for
    idx / out / lse, then timed pisa_bsa_bwd calls.  One JSON line.  Not the bench line."""
    import torch

    import paper_2609_31093_b200 as P
    from paper_2609_31093_b200 import binding as PB

    torch.cuda.set_device(0)
    try:
        peaks = json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except Exception:
        peaks = {}
    tens_peak = peaks.get("bf16_tflops_sustained", 1400.0)
    w = get_workload(args.workload)
    t = S.make_inputs(w)
    p = P.Params.from_workload(w)
    dev = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).cuda()
    q, k, v = dev(t["q"]), dev(t["k"]), dev(t["v"])
    pyramid = PB.alloc_pyramid(p)
    idx = torch.empty((w.B, w.Hkv, w.N, w.K), dtype=torch.int32, device="cuda")
    out = torch.empty_like(q)
    lse = torch.empty((w.B, w.Hq, w.N), dtype=torch.float32, device="cuda")
    ws = PB.alloc_workspace(p, PB.OP_FORWARD)
    P.pisa_forward(p, q, k, v, pyramid, idx, out, lse, ws)
    torch.cuda.synchronize()
    del ws
    gen = torch.Generator(device="cuda").manual_seed(77)
    dout = torch.randn(q.shape, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    dq, dk, dv = torch.empty_like(q), torch.empty_like(k), torch.empty_like(v)
    wsb = PB.alloc_workspace(p, PB.OP_BSA_BWD)
    P.set_forward_chunks(args.forward_chunks)
    for _ in range(max(1, args.warmup)):
        P.pisa_bsa_bwd(p, q, k, v, idx, out, lse, dout, dq, dk, dv, wsb)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        P.pisa_bsa_bwd(p, q, k, v, idx, out, lse, dout, dq, dk, dv, wsb)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    # per-kernel times: one more call with every kernel alone on the GPU (a large backward runs as
    # chunks on two streams, as the forward does)
    P.set_forward_chunks(1)
    P.set_stage_timing(True)
    P.pisa_bsa_bwd(p, q, k, v, idx, out, lse, dout, dq, dk, dv, wsb)
    kern = P.get_kernel_ms()
    P.set_stage_timing(False)
    P.set_forward_chunks(args.forward_chunks)
    wc = work_counts(w)
    flops = 2.5 * wc["attn_flops"]                     # five products of the forward's two shapes
    t_tiles = kern.get("backward_tiles", ms)
    row = {"backward": describe(w), "ms_per_call": ms, "tokens_per_s": w.B * w.N / (ms * 1e-3), "kernels_ms": kern,
           "kernels_ms_note": "each kernel alone (chunking off); ms_per_call is the chunked call",
           "algorithmic_tflop": flops / 1e12,
           "roofline": {"kernel": "backward_tiles", "bound": "tensor", "achieved": flops / (t_tiles * 1e-3) / 1e12,
                        "peak": tens_peak, "unit": "TFLOP/s", "frac": flops / (t_tiles * 1e-3) / 1e12 / tens_peak},
           "status": P.read_status(wsb)}
    print(json.dumps(row), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg4")
    ap.add_argument("--path", default="auto", choices=["auto", "simt", "tensor"])
    ap.add_argument("--ref-queries", type=int, default=4096,
                    help="sampled query positions the CPU oracle is timed on (all cores; a quarter of them on one core)")
    ap.add_argument("--no-parity", action="store_true", help="skip the oracle check of the timed buffers")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--forward-chunks", type=int, default=0,
                    help="upper limit on the chunks pisa_forward runs on two streams (0 = automatic, 1 = never split; "
                         "1 is what a per-kernel ncu capture wants)")
    ap.add_argument("--sweep", action="store_true", help="routing latency vs N and the flat selector (not the bench line)")
    ap.add_argument("--backward", action="store_true", help="attention backward with frozen indices (not the bench line)")
    ap.add_argument("--quality", action="store_true", help="Recall@K / MassRatio of the score modes vs full attention (not the bench line)")
    ap.add_argument("--decode", action="store_true", help="decoding latency vs context length (not the bench line)")
    args = ap.parse_args()
    if args.sweep:
        run_sweep(args)
        return
    if args.decode:
        run_decode(args)
        return
    if args.quality:
        run_quality(args)
        return
    if args.backward:
        run_backward(args)
        return
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

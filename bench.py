#!/usr/bin/env python
"""Benchmark of the DISCO logit tails on B200.

A step is one speculative iteration of the hot path: draft steps (LM head, soft-max statistics,
top-10 / entropy / position features, halt classifier, stopping rule) until the classifier or SL_max
stops the drafting, then one verification (LM head on SL+1 rows, greedy tokens, accepted prefix, bonus).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload vicuna_b1] [--impl ours|reference]

Rank 0 prints one JSON line.  With N > 1 every rank runs an independent replica (the path does not
shard); the value is the sum over replicas divided by the slowest replica's time.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2405_04304_b200 import inputs  # noqa: E402

METRIC = "draft-step+verify iterations/sec"
UNIT = "iterations/s"
L2_BYTES = 126 * 1024 * 1024


def measured_peaks():
    """(HBM GB/s, sustained bf16 TFLOP/s, 'measured' | 'fallback')."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            j = json.load(f)
        return float(j["hbm_gbs"]), float(j.get("bf16_tflops_sustained", 1400.0)), "measured"
    return 6650.0, 1400.0, "fallback"


# ------------------------------------------------------------------------------------------ ncu traffic
# dram__bytes_read.sum + dram__bytes_write.sum per launch, from the ncu captures summarised under
# profiles/.  Valid only for the kernel sources they were taken on: reported as null once csrc/ changes.
NCU_TRAFFIC = {
    "sources": "347370975812aea5",
    "bytes_per_launch": {
        ("vicuna_b1", "verification tail"): 327.77e6 + 4.34e6,
        ("vicuna_b1", "draft-step tail"): 49.23e6 + 0.02e6,
    },
}


def kernel_sources_hash() -> str:
    import glob
    import hashlib
    h = hashlib.sha256()
    for f in sorted(glob.glob(os.path.join(ROOT, "paper_2405_04304_b200", "csrc", "*"))):
        with open(f, "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def ncu_traffic(workload: str, kernel: str):
    if kernel_sources_hash() != NCU_TRAFFIC["sources"]:
        return None
    return NCU_TRAFFIC["bytes_per_launch"].get((workload, kernel))


# ------------------------------------------------------------------------------------------ ranks
def max_over_ranks(values, device="cpu"):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group).
    Every rank times its own replica; the job is as slow as its slowest replica."""
    if not (torch.distributed.is_available() and torch.distributed.is_initialized()):
        return [float(v) for v in values]
    t = torch.tensor([float(v) for v in values], dtype=torch.float64, device=device)
    torch.distributed.all_reduce(t, op=torch.distributed.ReduceOp.MAX)
    return [float(v) for v in t.cpu()]


def replica_seed(workload_seed: int, rank: int) -> int:
    """Each rank runs an independent replica of the workload on its own seeded inputs."""
    return workload_seed + 1000 * rank


def whole_job_value(steps_per_rank: int, world: int, seconds: float) -> float:
    """Iterations per second of the whole job: all replicas' steps over the slowest replica's time."""
    return steps_per_rank * world / seconds


# ------------------------------------------------------------------------------------------ clocks
class ClockSampler:
    """Polls SM clock and throttle reasons through NVML while the timed region runs (read-only)."""

    def __init__(self, index: int, period_s: float = 0.004):
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self.period = period_s
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksEventReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
        }
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self.nv is not None:
            self._thread = threading.Thread(target=self._loop, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        med = int(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------------------ workload
class Data:
    """All seeded inputs of T iterations of a workload, resident on the device (and, for the
    end-to-end leg, in pinned host memory)."""

    def __init__(self, wl: inputs.Workload, T: int, seed: int, device: str):
        self.wl, self.T = wl, T
        B, S = wl.B, wl.sl_max
        self.n_rot = max(2, -(-2 * L2_BYTES // (wl.V * wl.d_D * 2)) + 1)   # copies of W_D: > 2x L2 in total
        W_D = inputs.lm_head(wl.V, wl.d_D, inputs.sub_seed(seed, 1), device=device)
        self.W_D = [W_D] + [W_D.clone() for _ in range(self.n_rot - 1)]
        self.W_T = inputs.lm_head(wl.V, wl.d_T, inputs.sub_seed(seed, 2), device=device)
        self.clf_params = inputs.classifier_params(wl.H, inputs.sub_seed(seed, 3))
        # distinct iterations held in memory (cycled if T is larger)
        per_it = B * (S * wl.d_D + (S + 1) * wl.d_T) * 2
        self.n_distinct = int(max(1, min(T, (3 << 30) // per_it)))
        D = self.n_distinct
        self.h_D = inputs.hidden(D * S * B, wl.d_D, inputs.sub_seed(seed, 4), device=device).view(D, S, B, wl.d_D)
        self.H_T = inputs.hidden(D * B * (S + 1), wl.d_T, inputs.sub_seed(seed, 5), device=device).view(
            D, B * (S + 1), wl.d_T)
        # draft ids offered to verification: the target's greedy tokens, corrupted per position.
        # (Harness-side fp32 matmul; any ids are valid inputs, the kernels are timed on whatever they get.)
        Wf = self.W_T.float()
        tgt = torch.empty((D, B * (S + 1)), dtype=torch.int32)
        rows = self.H_T.view(-1, wl.d_T)
        flat = torch.empty(rows.shape[0], dtype=torch.int64, device=device)
        for r0 in range(0, rows.shape[0], 2048):
            flat[r0:r0 + 2048] = (rows[r0:r0 + 2048].float() @ Wf.T).argmax(-1)
        del Wf
        tgt.copy_(flat.view(D, B * (S + 1)).to(torch.int32).cpu())
        clean = tgt.view(D, B, S + 1)[:, :, :S].contiguous()
        if wl.accept_beta is not None:
            alpha = inputs.beta_rates(B, wl.accept_beta[0], wl.accept_beta[1], inputs.sub_seed(seed, 6))
            p = (1.0 - alpha).view(1, B, 1).expand(D, B, S)
        else:
            p = wl.p_corrupt
        self.draft_full = inputs.corrupt_ids(clean, p, wl.V, inputs.sub_seed(seed, 7))      # [D, B, S] cpu
        if wl.sl_mode == "uniform":
            self.forced_sl = inputs.uniform_sl(D * B, 1, S, inputs.sub_seed(seed, 8)).view(D, B)
        else:
            self.forced_sl = None

    def idx(self, it: int) -> int:
        return it % self.n_distinct


def pack_iteration(data: Data, it: int, sl: np.ndarray):
    """Rows and draft ids of one verification for per-sequence look-aheads sl [B]."""
    wl = data.wl
    d = data.idx(it)
    sl_t = torch.as_tensor(sl, dtype=torch.int32)
    off = inputs.row_offsets(sl_t)
    if wl.B == 1:
        H = data.H_T[d, : int(sl[0]) + 1]
        ids = data.draft_full[d, 0, : int(sl[0])].contiguous()
    else:
        H = inputs.pack_rows(data.H_T[d], sl_t, wl.sl_max)
        ids = inputs.pack_ids(data.draft_full[d].reshape(-1), sl_t, wl.sl_max)
    return H, ids, off


# ------------------------------------------------------------------------------------------ our arm
def device_pass(ctx, data: Data, clf, wl, tau: float, Wm: int, K: int, stream, world: int, device, sampler=None):
    """Closed loop once (discovery + warm-up), then the same launches captured in CUDA graphs and timed.

    Returns the time of the K timed iterations, the times of graphs holding only their draft-step or
    only their verification launches, and the closed-loop trace."""
    B, S = wl.B, wl.sl_max
    T = Wm + K
    token = torch.zeros((T, S, B), dtype=torch.int32, device=device)
    conf = torch.zeros((T, S, B), dtype=torch.float32, device=device)
    halt = torch.zeros((T, S, B), dtype=torch.uint8, device=device)
    n_acc = torch.zeros((T, B), dtype=torch.int32, device=device)
    bonus = torch.zeros((T, B), dtype=torch.int32, device=device)
    pos_all = torch.zeros((T, S, B), dtype=torch.int32)
    act_all = torch.zeros((T, S, B), dtype=torch.uint8)
    nd_all = torch.arange(1, S + 1, dtype=torch.int32).view(S, 1).expand(S, B).contiguous().to(device)
    sl_all = np.zeros((T, B), dtype=np.int64)
    steps_all = np.zeros(T, dtype=np.int64)
    emitted = np.zeros(B, dtype=np.int64)
    packed = []
    rot = 0
    # ---------------- discovery: the closed loop, the host reads the halt flags ----------------
    with torch.cuda.stream(stream):
        for it in range(T):
            d = data.idx(it)
            active = np.ones(B, dtype=np.uint8)
            sl = np.zeros(B, dtype=np.int64)
            for j in range(S):
                pos_all[it, j] = torch.from_numpy((emitted + j + 1).astype(np.int32))
                act_all[it, j] = torch.from_numpy(active)
                pos_d = pos_all[it, j].to(device, non_blocking=False)
                act_d = act_all[it, j].to(device)
                ctx.draft_step(data.W_D[rot % data.n_rot], data.h_D[d, j], pos_d, nd_all[j], clf, tau, S,
                               token[it, j], conf[it, j], halt[it, j], active=act_d, stream=stream)
                rot += 1
                stream.synchronize()
                h = halt[it, j].cpu().numpy()
                sl[active == 1] = j + 1
                if data.forced_sl is not None:
                    stop = (data.forced_sl[d].numpy() <= j + 1)
                else:
                    stop = h.astype(bool)
                active = (active.astype(bool) & ~stop).astype(np.uint8)
                steps_all[it] = j + 1
                if not active.any():
                    break
            sl_all[it] = sl
            H, ids, off = pack_iteration(data, it, sl)
            ids_d, off_d = ids.to(device), off.to(device)
            packed.append((H, ids_d, off_d, int(off[-1])))
            ctx.verify_ragged(data.W_T, H, ids_d, off_d, B, int(off[-1]), n_acc[it], bonus[it], stream=stream)
            stream.synchronize()
            emitted += n_acc[it].cpu().numpy().astype(np.int64) + 1
    status = ctx.device_status()
    if status != 0:
        raise RuntimeError(f"device status {status} after the discovery pass")
    pos_dev, act_dev = pos_all.to(device), act_all.to(device)
    ref_token, ref_halt = token.clone(), halt.clone()
    ref_nacc, ref_bonus = n_acc.clone(), bonus.clone()

    # ---------------- the same launch sequence, captured in CUDA graphs ----------------
    timed = range(Wm, T)

    def enqueue(which: str):
        r = 0
        for it in timed:
            d = data.idx(it)
            if which in ("all", "draft"):
                for j in range(int(steps_all[it])):
                    ctx.draft_step(data.W_D[r % data.n_rot], data.h_D[d, j], pos_dev[it, j], nd_all[j], clf, tau,
                                   S, token[it, j], conf[it, j], halt[it, j], active=act_dev[it, j])
                    r += 1
            if which in ("all", "verify"):
                H, ids_d, off_d, R = packed[it]
                ctx.verify_ragged(data.W_T, H, ids_d, off_d, B, R, n_acc[it], bonus[it])

    graphs = {}
    launches = {}
    for which in ("all", "draft", "verify"):
        token.zero_(); halt.zero_(); n_acc.zero_(); bonus.zero_()
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        c0 = ctx.launch_count()
        with torch.cuda.graph(g, stream=stream):
            enqueue(which)
        launches[which] = ctx.launch_count() - c0
        graphs[which] = g

    def time_graph(g, smp=None):
        with torch.cuda.stream(stream):
            g.replay()                               # untimed replay (graph upload, caches, clocks)
            stream.synchronize()
            if world > 1:
                torch.distributed.barrier()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            if smp is not None:
                smp.__enter__()
            e0.record(stream)
            g.replay()
            e1.record(stream)
            stream.synchronize()
            torch.cuda.synchronize()
            if smp is not None:
                smp.__exit__()
            if world > 1:
                torch.distributed.barrier()
        return e0.elapsed_time(e1) * 1e-3

    t_all = time_graph(graphs["all"], sampler)
    # results of the replay must be those of the closed loop
    same = (torch.equal(token[Wm:], ref_token[Wm:]) and torch.equal(halt[Wm:], ref_halt[Wm:]) and
            torch.equal(n_acc[Wm:], ref_nacc[Wm:]) and torch.equal(bonus[Wm:], ref_bonus[Wm:]))
    if not same or ctx.device_status() != 0:
        raise RuntimeError("graph replay did not reproduce the closed-loop results")
    t_draft = time_graph(graphs["draft"])
    t_verify = time_graph(graphs["verify"])
    del graphs
    n_draft = int(steps_all[Wm:].sum())
    rows_total = int(sum(packed[it][3] for it in timed))
    return {"t_all": t_all, "t_draft": t_draft, "t_verify": t_verify, "n_draft": n_draft, "rows_total": rows_total,
            "sl_all": sl_all, "n_acc": ref_nacc.cpu().numpy(), "launches": launches["all"]}


def rooflines(wl, K: int, res: dict, hbm_peak: float, tensor_peak: float, peak_kind: str):
    """Achieved algorithmic GB/s (or, beyond the machine balance, TFLOP/s) of the two kernels against the
    measured peaks.  Returns (dominant kernel, other kernel)."""
    draft_bytes = res["n_draft"] * (wl.V * wl.d_D * 2 + wl.B * wl.d_D * 2)
    verify_bytes = K * wl.V * wl.d_T * 2 + res["rows_total"] * wl.d_T * 2
    verify_flops = 2.0 * res["rows_total"] * wl.V * wl.d_T
    roof_verify = {"kernel": "verification tail", "bound": "hbm", "achieved": verify_bytes / res["t_verify"] / 1e9,
                   "peak": hbm_peak, "peak_kind": peak_kind, "unit": "GB/s", "launches": K,
                   "avg_launch_us": res["t_verify"] / K * 1e6, "traffic": None,
                   "tensor_tflops": verify_flops / res["t_verify"] / 1e12}
    roof_draft = {"kernel": "draft-step tail", "bound": "hbm", "achieved": draft_bytes / res["t_draft"] / 1e9,
                  "peak": hbm_peak, "peak_kind": peak_kind, "unit": "GB/s", "launches": res["n_draft"],
                  "avg_launch_us": res["t_draft"] / max(res["n_draft"], 1) * 1e6, "traffic": None}
    for r in (roof_verify, roof_draft):
        r["traffic"] = ncu_traffic(wl.name, r["kernel"])
        r["frac"] = r["achieved"] / r["peak"]
        r["frac_of_nominal_8TBs"] = r["achieved"] / 8000.0
    if res["rows_total"] / K > tensor_peak * 1e12 / (hbm_peak * 1e9):   # rows per call beyond the machine balance
        roof_verify.update({"bound": "tensor", "hbm_gbs": roof_verify["achieved"],
                            "achieved": roof_verify["tensor_tflops"], "peak": tensor_peak, "unit": "TFLOP/s",
                            "frac": roof_verify["tensor_tflops"] / tensor_peak})
        roof_verify.pop("frac_of_nominal_8TBs")
    return (roof_verify, roof_draft) if res["t_verify"] >= res["t_draft"] else (roof_draft, roof_verify)


def run_ours(args, rank: int, world: int):
    from paper_2405_04304_b200 import binding, build
    build.build()
    dev_index = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(dev_index)
    device = f"cuda:{dev_index}"
    wl = inputs.WORKLOADS[args.workload]
    K, Wm = args.steps, args.warmup
    T = Wm + K
    data = Data(wl, T, replica_seed(wl.seed, rank), device)
    B, S = wl.B, wl.sl_max
    max_rows = B * (S + 1)
    ctx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=B, max_rows=max_rows, clf_hidden=wl.H)
    ctx.set_kernel_path(args.kernel_path)
    clf = binding.Classifier(*(t.to(device) for t in data.clf_params))
    stream = torch.cuda.Stream()
    hbm_peak, tensor_peak, peak_kind = measured_peaks()

    sampler = ClockSampler(dev_index)
    res = device_pass(ctx, data, clf, wl, wl.tau, Wm, K, stream, world, device, sampler)
    dominant, other = rooflines(wl, K, res, hbm_peak, tensor_peak, peak_kind)
    t_all = res["t_all"]

    # the same workload with the classifier overruled: tau = 0 never halts before SL_max (static SL)
    static = None
    if data.forced_sl is None and not args.no_static:
        Ks = min(K, 256)
        rs = device_pass(ctx, data, clf, wl, 0.0, Wm, Ks, stream, world, device)
        sd, so = rooflines(wl, Ks, rs, hbm_peak, tensor_peak, peak_kind)
        static = {"value": Ks * world / rs["t_all"], "unit": UNIT, "steps": Ks,
                  "mean_sl": float(rs["sl_all"][Wm:].mean()), "ms_per_step": rs["t_all"] / Ks * 1e3,
                  "roofline": sd, "roofline_other_kernel": so}

    # ---------------- end to end: host buffers through the *_host entry points, closed loop ----------
    e2e = run_e2e(ctx, data, clf, wl, Wm, K, stream, world)
    e2e["matches"] = all(np.array_equal(sl, res["sl_all"][it]) and np.array_equal(na, res["n_acc"][it])
                         for it, (sl, na) in enumerate(e2e["trace"]))

    t_all, e2e["seconds"] = max_over_ranks([t_all, e2e["seconds"]], device)

    out = {
        "metric": METRIC, "value": whole_job_value(K, world, t_all), "unit": UNIT, "n_gpus": world, "steps": K, "warmup": Wm,
        "ms_per_step": t_all / K * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16 inputs, fp32 accumulate", "data": "synthetic (seeded Gaussian LM heads and hidden states)",
        "config": {"workload": wl.name, "V": wl.V, "d_draft": wl.d_D, "d_target": wl.d_T, "batch": B,
                   "sl_max": S, "tau": wl.tau, "clf_hidden": wl.H, "p_corrupt": wl.p_corrupt,
                   "sl_source": wl.sl_mode, "mean_sl": float(res["sl_all"][Wm:].mean()),
                   "mean_accepted": float(res["n_acc"][Wm:].mean()),
                   "draft_steps_per_iteration": res["n_draft"] / K, "replicas": world,
                   "l2": f"draft LM head rotates through {data.n_rot} copies (> 2x L2); the target LM head alone "
                         "exceeds L2", "launch": "CUDA graph of the K iterations' kernels"},
        "roofline": dominant, "roofline_other_kernel": other,
        "e2e": {"value": whole_job_value(K, world, e2e["seconds"]), "unit": UNIT, "h2d_bytes_per_step": e2e["h2d"] / K,
                "d2h_bytes_per_step": e2e["d2h"] / K, "matches_device_run": e2e["matches"]},
        "gpu_launches": res["launches"], "clocks": sampler.summary(),
    }
    if static is not None:
        out["static_sl_max"] = static
    if wl.B == 1 and not args.no_static:
        out["other_modes"] = other_modes(ctx, data, clf, wl, stream, device)
        if ctx.device_status() != 0:
            raise RuntimeError(f"device status {ctx.device_status()} after the other modes")
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        out["cpu_baseline"] = cpu_baseline(data, wl, budget_s=args.cpu_seconds)
    ctx.close()
    return out


def other_modes(ctx, data: Data, clf, wl, stream, device) -> dict:
    """Average device time of the further entry points on the same inputs (one sequence, look-ahead
    SL_max), each as a CUDA-graph replay of 20 calls with the draft LM head rotating: the draft step with
    the perplexity rule, the sampled draft step, verification with sampling, and bulk feature extraction."""
    B, S, V = wl.B, wl.sl_max, wl.V
    R = B * (S + 1)
    g = torch.Generator(device=device).manual_seed(12345)
    u = torch.rand(B, generator=g, device=device)
    ua = torch.rand(B * S, generator=g, device=device)
    us = torch.rand(B, generator=g, device=device)
    pos = torch.ones(B, dtype=torch.int32, device=device)
    nd = torch.ones(B, dtype=torch.int32, device=device)
    tok = torch.zeros(B, dtype=torch.int32, device=device)
    conf = torch.zeros(B, device=device)
    halt = torch.zeros(B, dtype=torch.uint8, device=device)
    nll = torch.zeros(B, device=device)
    ptok = torch.zeros(B, device=device)
    dprobs = torch.zeros(S, B, V, device=device)
    yT = torch.zeros(R, V, device=device)
    ids = data.draft_full[0].reshape(-1).to(device)
    na = torch.zeros(B, dtype=torch.int32, device=device)
    nx = torch.zeros(B, dtype=torch.int32, device=device)
    N = 256                                        # positions of the feature-extraction pass
    HD = data.h_D.reshape(-1, wl.d_D)
    HT = data.H_T.reshape(-1, wl.d_T)
    N = min(N, HD.shape[0], HT.shape[0])
    from paper_2405_04304_b200 import binding
    fx = binding.Context(wl.V, wl.d_D, wl.d_T, max_batch=B, max_rows=N, clf_hidden=wl.H)   # scratch for N rows
    fD = torch.zeros(N, 12, device=device); fT = torch.zeros(N, 12, device=device)
    tv = torch.zeros(N, device=device); lab = torch.zeros(N, dtype=torch.uint8, device=device)
    tD = torch.zeros(N, dtype=torch.int32, device=device); tT = torch.zeros(N, dtype=torch.int32, device=device)
    yDn = torch.zeros(N, V, device=device); yTn = torch.zeros(N, V, device=device)
    posN = torch.arange(N, dtype=torch.int32, device=device)
    h = data.h_D[0, 0]
    H_T = data.H_T[0]
    calls = {
        "draft_step_ppl": lambda i: ctx.draft_step_ppl(data.W_D[i % data.n_rot], h, nd, nll, 1e9, S, tok, conf, halt,
                                                       stream=stream),
        "draft_step_sample": lambda i: ctx.draft_step_sample(data.W_D[i % data.n_rot], h, pos, nd, clf, wl.tau, S, u,
                                                             tok, conf, halt, dprobs[i % S], p_token=ptok,
                                                             stream=stream),
        "verify_sample": lambda i: ctx.verify_sample_ragged(data.W_T, H_T, ids, dprobs, None, B, R, ua, us, na, nx, yT,
                                                            stream=stream),
        "extract_features": lambda i: fx.extract_features(data.W_D[i % data.n_rot], HD[:N], data.W_T, HT[:N], posN,
                                                           fD, fT, tv, lab, tD, tT, yDn, yTn, stream=stream),
    }
    out = {}
    reps = 20
    e0 = torch.cuda.Event(enable_timing=True)
    e1 = torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        for name, fn in calls.items():
            for i in range(3):
                fn(i)
            stream.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for i in range(reps):
                    fn(i)
            graph.replay()
            stream.synchronize()
            e0.record(stream)
            graph.replay()
            e1.record(stream)
            stream.synchronize()
            out[name + "_us"] = e0.elapsed_time(e1) * 1e3 / reps
    if fx.device_status() != 0:
        raise RuntimeError(f"device status {fx.device_status()} after feature extraction")
    fx.close()
    out["extract_features_positions"] = N
    out["look_ahead"] = S
    return out


def run_e2e(ctx, data: Data, clf, wl, Wm: int, K: int, stream, world: int):
    """Closed loop through the host-buffer entry points: per-step inputs start in pinned host memory,
    every result (halt flag, token, accepted length, bonus) is read back by the host."""
    B, S = wl.B, wl.sl_max
    D = data.n_distinct
    h_D_host = data.h_D.cpu().pin_memory()
    H_T_host = data.H_T.cpu().pin_memory()
    token = torch.zeros(B, dtype=torch.int32).pin_memory()
    conf = torch.zeros(B, dtype=torch.float32).pin_memory()
    halt = torch.zeros(B, dtype=torch.uint8).pin_memory()
    n_acc = torch.zeros(B, dtype=torch.int32).pin_memory()
    bonus = torch.zeros(B, dtype=torch.int32).pin_memory()
    pos = torch.zeros(B, dtype=torch.int32).pin_memory()
    nd = torch.zeros(B, dtype=torch.int32).pin_memory()
    act = torch.ones(B, dtype=torch.uint8).pin_memory()
    h2d = d2h = 0
    emitted = np.zeros(B, dtype=np.int64)
    trace = []
    rot = 0
    # numpy views of the pinned buffers: the loop's own bookkeeping stays off torch's dispatcher
    pos_np, nd_np, act_np, halt_np, nacc_np = pos.numpy(), nd.numpy(), act.numpy(), halt.numpy(), n_acc.numpy()
    forced = None if data.forced_sl is None else data.forced_sl.numpy()
    off = torch.zeros(B + 1, dtype=torch.int32).pin_memory()
    off_np = off.numpy()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for it in range(Wm + K):
        if it == Wm:
            torch.cuda.synchronize()
            if world > 1:
                torch.distributed.barrier()
            e0.record(stream)
            h2d = d2h = 0
        d = data.idx(it)
        act_np[:] = 1
        sl = np.zeros(B, dtype=np.int64)
        for j in range(S):
            pos_np[:] = emitted + (j + 1)
            nd_np[:] = j + 1
            ctx.draft_step_host(data.W_D[rot % data.n_rot], h_D_host[d, j], pos, nd, clf, wl.tau, S, token, conf,
                                halt, active=act if B > 1 else None, stream=stream)
            rot += 1
            h2d += B * (wl.d_D * 2 + 4 + 4 + 1)
            a = act_np.astype(bool)
            d2h += int(a.sum()) * (4 + 4 + 1)
            sl[a] = j + 1
            stop = (forced[d] <= j + 1) if forced is not None else halt_np.astype(bool)
            act_np[:] = a & ~stop
            if not act_np.any():
                break
        sl_t = torch.as_tensor(sl, dtype=torch.int32)
        off_np[1:] = np.cumsum(sl + 1)
        if B == 1:
            H = H_T_host[d, : int(sl[0]) + 1]
            ids = data.draft_full[d, 0, : int(sl[0])].contiguous()
        else:
            H = inputs.pack_rows(H_T_host[d], sl_t, S)
            ids = inputs.pack_ids(data.draft_full[d].reshape(-1), sl_t, S)
        R = int(off_np[-1])
        ctx.verify_ragged_host(data.W_T, H, ids if ids.numel() else None, off, B, R, n_acc, bonus, stream=stream)
        h2d += R * wl.d_T * 2 + (R - B) * 4 + (B + 1) * 4
        d2h += B * 8
        emitted += nacc_np.astype(np.int64) + 1
        trace.append((sl.copy(), nacc_np.copy()))
    e1.record(stream)
    torch.cuda.synchronize()
    if world > 1:
        torch.distributed.barrier()
    return {"seconds": e0.elapsed_time(e1) * 1e-3, "h2d": h2d, "d2h": d2h, "matches": True, "trace": trace}


# ------------------------------------------------------------------------------------------ CPU legs
def oracle_iteration(oracle, wl, W_D, W_T, clf, h_D, H_T, draft, emitted, nthreads, forced_sl=None):
    """One iteration with the CPU oracle (closed loop on its own halt flags).  Arrays are numpy."""
    B, S = wl.B, wl.sl_max
    active = np.ones(B, dtype=np.uint8)
    sl = np.zeros(B, dtype=np.int64)
    for j in range(S):
        res = oracle.draft_step(W_D, h_D[j], (emitted + j + 1).astype(np.int32), np.full(B, j + 1, np.int32), clf,
                                wl.tau, S, active=active, nthreads=nthreads)
        sl[active == 1] = j + 1
        stop = (forced_sl <= j + 1) if forced_sl is not None else (res.halt == 1)
        active = (active.astype(bool) & ~stop).astype(np.uint8)
        if not active.any():
            break
    sl_t = torch.as_tensor(sl, dtype=torch.int32)
    off = inputs.row_offsets(sl_t).numpy()
    rows = np.concatenate([H_T[b * (S + 1): b * (S + 1) + sl[b] + 1] for b in range(B)])
    ids = np.concatenate([draft[b, : sl[b]] for b in range(B)]).astype(np.int32)
    v = oracle.verify_ragged(W_T, rows, ids, off, nthreads=nthreads)
    return emitted + v.n_accept + 1


def cpu_baseline(data: Data, wl, budget_s: float):
    """The oracle, as it stands, on the host cores: whole iterations of the same workload until the
    time budget is used (at least two)."""
    import oracle
    oracle.build()
    cores = oracle.hardware_threads()
    W_D, W_T = inputs.bf16_bits(data.W_D[0]), inputs.bf16_bits(data.W_T)
    W1, b1, w2, b2 = data.clf_params
    clf = oracle.Classifier(W1.numpy(), b1.numpy(), w2.numpy(), b2.numpy())
    emitted = np.zeros(wl.B, dtype=np.int64)
    n, t0 = 0, time.perf_counter()
    while n < 2 or (time.perf_counter() - t0 < budget_s and n < data.n_distinct):
        d = data.idx(n)
        h_D = inputs.bf16_bits(data.h_D[d].reshape(-1, wl.d_D)).reshape(wl.sl_max, wl.B, wl.d_D)
        H_T = inputs.bf16_bits(data.H_T[d])
        forced = data.forced_sl[d].numpy() if data.forced_sl is not None else None
        emitted = oracle_iteration(oracle, wl, W_D, W_T, clf, h_D, H_T, data.draft_full[d].numpy(), emitted, cores,
                                   forced)
        n += 1
    dt = time.perf_counter() - t0
    return {"value": n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": f"first {n} iterations of {wl.name} (all vocabulary rows), {dt:.1f} s"}


def run_reference(args):
    """--impl reference: the CPU oracle timed on the host cores.  Each step is one iteration of the
    workload restricted to the first V_s vocabulary rows of both LM heads (V_s chosen so that the whole
    run takes about two minutes); the time of a step is scaled by V / V_s."""
    import oracle
    oracle.build()
    wl = inputs.WORKLOADS[args.workload]
    K, Wm = args.steps, args.warmup
    cores = oracle.hardware_threads()
    W1, b1, w2, b2 = inputs.classifier_params(wl.H, inputs.sub_seed(wl.seed, 3))
    clf = oracle.Classifier(W1.numpy(), b1.numpy(), w2.numpy(), b2.numpy())
    # calibrate on 1024 rows
    Vc = min(wl.V, 1024)
    Wc = inputs.bf16_bits(inputs.lm_head(Vc, wl.d_T, 1))
    Hc = inputs.bf16_bits(inputs.hidden(wl.B * (wl.sl_max + 1), wl.d_T, 2))
    t0 = time.perf_counter()
    oracle.project(Wc, Hc, nthreads=cores)
    per_row = (time.perf_counter() - t0) / Vc * 1.5          # + draft steps
    budget = args.reference_seconds / max(1, K + Wm)
    Vs = int(max(64, min(wl.V, budget / per_row)))
    W_D = inputs.bf16_bits(inputs.lm_head(Vs, wl.d_D, inputs.sub_seed(wl.seed, 1)))
    W_T = inputs.bf16_bits(inputs.lm_head(Vs, wl.d_T, inputs.sub_seed(wl.seed, 2)))
    sub = wl.with_(V=Vs)
    emitted = np.zeros(wl.B, dtype=np.int64)
    total = 0.0
    rng = np.random.default_rng(wl.seed)
    for it in range(Wm + K):
        h_D = inputs.bf16_bits(inputs.hidden(wl.sl_max * wl.B, wl.d_D, inputs.sub_seed(wl.seed, 4, it))).reshape(
            wl.sl_max, wl.B, wl.d_D)
        H_T = inputs.bf16_bits(inputs.hidden(wl.B * (wl.sl_max + 1), wl.d_T, inputs.sub_seed(wl.seed, 5, it)))
        draft = rng.integers(0, Vs, size=(wl.B, wl.sl_max)).astype(np.int32)
        forced = None
        if wl.sl_mode == "uniform":
            forced = inputs.uniform_sl(wl.B, 1, wl.sl_max, inputs.sub_seed(wl.seed, 8, it)).numpy()
        t0 = time.perf_counter()
        emitted = oracle_iteration(oracle, sub, W_D, W_T, clf, h_D, H_T, draft, emitted, cores, forced)
        if it >= Wm:
            total += time.perf_counter() - t0
    scaled = total * (wl.V / Vs)
    val = K / scaled
    sample = f"each step: one iteration on the first {Vs} of {wl.V} vocabulary rows, time scaled by {wl.V / Vs:.1f}"
    return {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": K,
            "warmup": Wm, "ms_per_step": scaled / K * 1e3, "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": "f64", "data": "synthetic (seeded Gaussian LM heads and hidden states)",
            "config": {"workload": wl.name, "V": wl.V, "d_draft": wl.d_D, "d_target": wl.d_T, "batch": wl.B,
                       "sl_max": wl.sl_max, "tau": wl.tau},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1024)
    ap.add_argument("--warmup", type=int, default=8)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vicuna_b1", choices=sorted(inputs.WORKLOADS))
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    ap.add_argument("--reference-seconds", type=float, default=120.0)
    ap.add_argument("--kernel-path", type=int, default=0, help="0 automatic; 1..3 force a kernel family (tuning)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-static", action="store_true", help="skip the extra pass with SL forced to SL_max")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3)
    rank = int(os.environ.get("RANK", 0))
    world = int(os.environ.get("WORLD_SIZE", 1))

    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        torch.cuda.set_device(int(os.environ.get("LOCAL_RANK", 0)))
        torch.distributed.init_process_group("nccl")
    out = run_ours(args, rank, world)
    if rank == 0:
        print(json.dumps(out), flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


if __name__ == "__main__":
    main()

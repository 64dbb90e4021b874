#!/usr/bin/env python
"""Benchmark of the fused credit-assignment scans on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--no-sweep]

A "step" is one pass of the whole hot path over one synthetic batch: the seven algorithms (GAE,
V-Trace, Retrace, TD(lambda), discounted returns, eligibility trace, episodic prefix sum), one fused
kernel launch each, on the 16384 x 2048 bandwidth-saturating configuration with per-step truncation
handling.  `value` counts N*T env-steps per algorithm pass, i.e. 7*N*T per step and per GPU.

Rank 0 prints one JSON line per detail record (per-algorithm figures, extension entry points, the
cold-L2 cases of the smaller configurations) and LAST the headline line, which is kept below 2 KB and
holds every key of the bench contract (value, roofline, cpu_baseline, e2e, clocks).  With N > 1 (torchrun) every rank works on its own batch of the same
shape (rows are independent: weak scaling, no collective on the data path); the time is the max
over ranks.  `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import os
import re
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np

METRIC = "env-steps/s"
ALGOS = ("gae", "vtrace", "retrace", "td_lambda", "discounted_return", "elig_trace", "episodic_prefix_sum")
WORKLOAD = dict(N=16384, T=2048)
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per launch on the bench workload come from a committed
# one-pass ncu capture of the full-size run: `--traffic-from-ncu` turns ncu's CSV log into this file,
# keyed by algorithm with the kernel instance beside each figure.
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "dram_traffic_16384x2048.json")
HEADLINE_LIMIT = 2048        # the headline (last stdout line) stays below this many bytes


# --------------------------------------------------------------------------------------------- helpers
def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def algorithmic_bytes(ro, algo: str) -> int:
    """Compulsory input + output bytes of one launch: every [N,T] input read once, every output
    written once, the [N] bootstrap once, and of the 2-D truncation bootstrap only the 32-byte
    sectors that hold a value the kernel must read (truncated and not terminated)."""
    S = ro.N * ro.T
    f32_in = {"gae": 2, "vtrace": 3, "retrace": 4, "td_lambda": 2, "discounted_return": 1,
              "elig_trace": 1, "episodic_prefix_sum": 1}[algo]
    f32_out = {"gae": 2, "vtrace": 2}.get(algo, 1)
    b = 4 * S * (f32_in + f32_out) + S                      # fp32 tensors + the done mask
    if algo not in ("elig_trace", "episodic_prefix_sum"):
        b += 4 * ro.N                                       # window-edge bootstrap
        if ro.truncs is not None:
            b += S                                          # truncation mask
            idx = np.flatnonzero((ro.truncs.ravel() != 0) & (ro.dones.ravel() == 0))
            b += 32 * int(np.unique(idx // 8).size)
    return int(b)


def kernel_instance(binding, algo: str, has_truncs: bool, N: int, T: int) -> str:
    """Name of the kernel instance a call on whole tiles takes, as ncu prints it: template arguments are
    (algorithm id, truncation handling, vector accesses, threads, steps per thread, blocks per SM, row-aligned tiling)."""
    tr = bool(has_truncs) and algo not in ("elig_trace", "episodic_prefix_sum")
    vi = binding.rlcs_debug_variant_for(algo, tr, N, T)
    kname = "scan_kernel_tma" if vi["ring_stages"] else "scan_kernel"
    args = f"{binding.ALGORITHM_IDS[algo]},{int(tr)},1,{vi['threads']},{vi['steps_per_thread']},{vi['blocks_per_sm']}"
    return f"{kname}<{args}>" if vi["ring_stages"] else f"{kname}<{args},0>"       # last argument: not the row-aligned instantiation


def load_traffic(path: str = TRAFFIC_JSON) -> dict:
    try:
        with open(path) as fh:
            return json.load(fh).get("kernels", {})
    except Exception:
        return {}


def traffic_for(algo: str, instance: str, table: dict):
    """Captured DRAM bytes per launch of `algo`, or None when the capture was taken on another kernel
    instance than the one that runs now (a stale figure is worse than none)."""
    rec = table.get(algo)
    if not rec or rec.get("kernel") != instance:
        return None
    return int(rec["dram_bytes_per_launch"])


def traffic_from_ncu(csv_path: str, out_path: str = TRAFFIC_JSON, command: str = "") -> dict:
    """Turn the CSV log of `ncu --metrics dram__bytes_read.sum,dram__bytes_write.sum --csv` over the
    bench command into the committed traffic table: per algorithm the kernel instance and the mean of
    read + write bytes over its captured launches."""
    import csv
    ids = {0: "gae", 1: "td_lambda", 2: "discounted_return", 3: "vtrace", 4: "retrace", 5: "elig_trace",
           6: "episodic_prefix_sum"}
    unit = {"byte": 1.0, "Kbyte": 1e3, "Mbyte": 1e6, "Gbyte": 1e9}
    with open(csv_path, newline="") as fh:
        lines = [ln for ln in fh if ln.startswith('"')]
    per_launch = {}                                   # launch id -> [kernel, bytes]
    for row in csv.DictReader(lines):
        name = row["Kernel Name"]
        if "dram__bytes" not in row["Metric Name"]:
            continue
        val = float(row["Metric Value"].replace(",", "")) * unit.get(row["Metric Unit"], 1.0)
        rec = per_launch.setdefault(row["ID"], [name, 0.0])
        rec[1] += val
    by_kernel = {}
    for name, b in per_launch.values():
        by_kernel.setdefault(name, []).append(b)
    kernels = {}
    for name, vals in by_kernel.items():
        m = re.search(r"(scan_kernel\w*)\s*<([^>]*)>", name)
        if m is None or m.group(1) not in ("scan_kernel", "scan_kernel_tma"):
            continue
        targs = [a.strip().replace("(rlcs::Algo)", "").replace("(bool)", "").replace("(int)", "") for a in m.group(2).split(",")]
        targs = ["1" if a == "true" else "0" if a == "false" else a for a in targs]
        algo = ids.get(int(targs[0]))
        if algo is None:
            continue
        short = f"{m.group(1)}<{','.join(targs)}>"
        kernels[algo] = {"kernel": short, "launches": len(vals), "dram_bytes_per_launch": int(round(sum(vals) / len(vals)))}
    doc = {"workload": f"num_envs={WORKLOAD['N']}, T={WORKLOAD['T']}, truncation handling on", "command": command,
           "metrics": "dram__bytes_read.sum + dram__bytes_write.sum, mean over the captured launches", "kernels": kernels}
    with open(out_path, "w") as fh:
        json.dump(doc, fh, indent=1)
        fh.write("\n")
    return doc


def build_headline(*, value, world, steps, warmup, ms_per_step, workload, clocks, e2e, launches, roofline,
                   cpu_baseline=None, per_algorithm_frac=None, small_frac=None, detail_file=None) -> dict:
    """The last stdout line: every key the bench contract names and nothing bulky.  Per-algorithm,
    extension and sweep figures are printed before it, one JSON line each."""
    line = {
        "metric": METRIC, "value": value, "unit": METRIC, "n_gpus": world, "steps": steps, "warmup": warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": {"workload": workload, "l2": "inputs larger than L2, no flush"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "roofline": roofline,
    }
    if cpu_baseline is not None:
        line["cpu_baseline"] = cpu_baseline
    if per_algorithm_frac:
        line["frac_of_peak"] = per_algorithm_frac
    if small_frac:
        line["small_configs_frac_of_peak"] = small_frac
    if detail_file:
        line["detail_file"] = detail_file
    return line


def emit(details: list, headline: dict, detail_file=None):
    """Detail lines first, the headline last and alone on the final line."""
    text = json.dumps(headline)
    for drop in ("small_configs_frac_of_peak", "frac_of_peak"):        # never let the headline outgrow the limit
        if len(text) < HEADLINE_LIMIT:
            break
        headline.pop(drop, None)
        text = json.dumps(headline)
    assert len(text) < HEADLINE_LIMIT, f"headline line is {len(text)} bytes"
    if detail_file:
        with open(detail_file, "w") as fh:
            json.dump({"headline": headline, "details": details}, fh, indent=1)
    for d in details:
        print(json.dumps(d), flush=True)
    print(text, flush=True)


class ClockSampler:
    """Samples SM clock and clock-event reasons through NVML while the timed region runs."""

    REASONS = {0x1: "gpu_idle", 0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown",
               0x10: "sync_boost", 0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown",
               0x80: "hw_power_brake_slowdown", 0x100: "display_clock_setting"}

    def __init__(self, index: int, period_s: float = 0.0005):
        self.samples, self.reasons, self.power = [], set(), []
        self.period, self._stop, self.max_mhz, self.ok = period_s, threading.Event(), None, False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.ok = False
        self.t = threading.Thread(target=self._run, daemon=True)

    def _once(self):
        nv = self.nv
        self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
        try:
            mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
        except Exception:
            mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
        for bit, name in self.REASONS.items():
            if mask & bit and name != "gpu_idle":
                self.reasons.add(name)
        try:
            self.power.append(nv.nvmlDeviceGetPowerUsage(self.h) / 1000.0)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                break
            time.sleep(self.period)

    def __enter__(self):
        if self.ok:
            self.t.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        if self.ok:
            self.t.join(timeout=2)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        return {"sm_mhz": int(statistics.median(self.samples)), "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples),
                "power_w_max": round(max(self.power), 1) if self.power else None}


# --------------------------------------------------------------------------------------------- GPU arm
class GpuBatch:
    """Device-resident inputs, outputs and workspace of one batch, and the seven calls on them."""

    NEEDS = {"gae": ("rewards", "values"), "vtrace": ("rewards", "values", "log_rhos"),
             "retrace": ("rewards", "q_sa", "expected_q", "log_rhos"), "td_lambda": ("rewards", "values"),
             "discounted_return": ("rewards",), "elig_trace": ("x", "any_done"), "episodic_prefix_sum": ("x", "any_done")}
    BACKWARD_COMMON = ("dones", "truncs", "trunc_bootstrap", "bootstrap")

    def __init__(self, ro, device, only=None):
        import torch
        from paper_2608_17641_b200 import binding as B
        self.B, self.ro, self.torch = B, ro, torch
        algos = ALGOS if only is None else (only,)
        keys = set()
        for a in algos:
            keys.update(self.NEEDS[a])
            if a not in ("elig_trace", "episodic_prefix_sum"):
                keys.update(self.BACKWARD_COMMON)
        src = lambda k: ro.any_done if k == "any_done" else getattr(ro, k)
        up = lambda a: None if a is None else torch.from_numpy(a).to(device, non_blocking=False)
        self.inp = {k: (up(src(k)) if k in keys else None) for k in ("rewards", "values", "q_sa", "expected_q", "log_rhos",
                                                                      "x", "dones", "truncs", "trunc_bootstrap", "bootstrap",
                                                                      "any_done")}
        new = lambda: torch.empty((ro.N, ro.T), dtype=torch.float32, device=device)
        self.out = {a: ((new(), new()) if a in ("gae", "vtrace") else new()) for a in algos}
        self.ws = B.Workspace(ro.N, ro.T, device=device)
        self.launches = 0

    def spec(self, algo: str):
        """(binding wrapper, positional arguments, keyword arguments) of one call."""
        B, i, o, p, ws = self.B, self.inp, self.out, self.ro.params, self.ws
        bw = (i["dones"], i["truncs"], i["trunc_bootstrap"], i["bootstrap"])
        if algo == "gae":
            return B.rlcs_gae, (i["rewards"], i["values"], *bw), dict(gamma=p["gamma"], lam=p["lam"], advantages=o[algo][0],
                                                                       returns=o[algo][1], workspace=ws)
        if algo == "vtrace":
            return B.rlcs_vtrace, (i["rewards"], i["values"], i["log_rhos"], *bw), dict(
                gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"], vs=o[algo][0], pg_advantages=o[algo][1], workspace=ws)
        if algo == "retrace":
            return B.rlcs_retrace, (i["rewards"], i["q_sa"], i["expected_q"], i["log_rhos"], *bw), dict(
                gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"], q_targets=o[algo], workspace=ws)
        if algo == "td_lambda":
            return B.rlcs_td_lambda, (i["rewards"], i["values"], *bw), dict(gamma=p["gamma"], lam=p["lam"], returns=o[algo], workspace=ws)
        if algo == "discounted_return":
            return B.rlcs_discounted_return, (i["rewards"], *bw), dict(gamma=p["gamma"], returns=o[algo], workspace=ws)
        if algo == "elig_trace":
            return B.rlcs_elig_trace, (i["x"], i["any_done"]), dict(gamma=p["gamma"], lam=p["lam"], traces=o[algo], workspace=ws)
        if algo == "episodic_prefix_sum":
            return B.rlcs_episodic_prefix_sum, (i["x"], i["any_done"]), dict(sums=o[algo], workspace=ws)
        raise KeyError(algo)

    def call(self, algo: str):
        fn, args, kwargs = self.spec(algo)
        fn(*args, **kwargs)
        self.launches += 1

    def prepared(self, algo: str):
        """The same call with its arguments marshalled once (binding.prepare)."""
        fn, args, kwargs = self.spec(algo)
        return self.B.prepare(fn, *args, **kwargs)

    def step(self, timed=None, events=None):
        """One pass of the seven calls.  `timed` = index of the one call of this step that is
        bracketed by the two CUDA events in `events` (on the launching stream)."""
        for k, a in enumerate(ALGOS):
            if k == timed:
                events[0].record()
            self.call(a)
            if k == timed:
                events[1].record()


def time_device(batch: GpuBatch, steps: int, warmup: int, dist):
    """K timed steps with inputs resident in HBM.  Per-kernel durations come from CUDA events on the
    launching stream inside the timed region: every step but the first brackets ONE of its seven
    launches (step k the launch (k-1) mod 7), so each kernel is sampled about K/7 times while the other
    six launches of a step run back to back as a caller would issue them -- an event between every pair
    of launches costs several per cent of a step by itself.  The first step brackets nothing: the
    stream is empty when the region starts, so an event recorded there would also time the host's
    launch latency.  Kernels that the timed region did not reach (K < 8) are sampled in extra, untimed
    steps.  The per-kernel figure is the median of its samples; a bracketed launch overlaps neither
    the kernel before it nor the one after it, so the figure includes its whole ramp-up and tail."""
    torch = batch.torch
    for _ in range(warmup):
        batch.step()
    n = len(ALGOS)
    extra = max(0, n + 1 - steps)
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps + extra)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    which = lambda k: (k - 1) % n if k > 0 else None
    dist.barrier()
    torch.cuda.synchronize()
    launches0 = batch.launches
    with ClockSampler(torch.cuda.current_device()) as clk:
        start.record()
        for k in range(steps):
            batch.step(which(k), ev[k])
        stop.record()
        torch.cuda.synchronize()
    dist.barrier()
    launches = batch.launches - launches0
    for k in range(steps, steps + extra):
        batch.step(which(k), ev[k])
    torch.cuda.synchronize()
    total_ms = start.elapsed_time(stop)
    per_algo_ms = {a: [ev[k][0].elapsed_time(ev[k][1]) for k in range(1, steps + extra) if which(k) == j]
                   for j, a in enumerate(ALGOS)}
    assert batch.ws.device_status() == 0, "device reported a carry-wait timeout"
    return total_ms, per_algo_ms, launches, clk.summary()


def time_gae_normalized(batch: GpuBatch, steps: int, peak: float):
    """Extension beyond the seven kernels: GAE + advantage normalisation (three launches) on the
    bench batch; algorithmic bytes = GAE's plus one read and one write of the advantages."""
    torch, B, ro = batch.torch, batch.B, batch.ro
    i, o, p = batch.inp, batch.out, ro.params
    ws = B.Workspace(ro.N, ro.T, nbytes=int(B.lib().rlcs_gae_normalized_workspace_bytes(ro.N, ro.T)))
    call = lambda: B.rlcs_gae_normalized(i["rewards"], i["values"], i["dones"], i["truncs"], i["trunc_bootstrap"],
                                         i["bootstrap"], gamma=p["gamma"], lam=p["lam"], eps=1e-8, ddof=1,
                                         advantages=o["gae"][0], returns=o["gae"][1], workspace=ws)
    for _ in range(3):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ab = algorithmic_bytes(ro, "gae") + 8 * ro.N * ro.T
    gbs = ab / (ms * 1e-3) / 1e9
    return {"ms": round(ms, 5), "launches_per_call": 3, "env_steps_per_s": ro.N * ro.T / (ms * 1e-3),
            "algorithmic_bytes": ab, "gbs": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4)}


def time_gae_skip(batch: GpuBatch, steps: int, peak: float, p_skip: float = 0.3):
    """Extension beyond the seven kernels: GAE with observation-skip masking (one launch, two scans per
    tile) on the bench batch with skip ~ Bernoulli(p_skip).  Algorithmic bytes = GAE's, plus the skip
    mask, plus one write of the filled values W (an output of the call)."""
    torch, B, ro = batch.torch, batch.B, batch.ro
    i, o, p = batch.inp, batch.out, ro.params
    g = torch.Generator(device="cuda").manual_seed(17641)
    skip = (torch.rand((ro.N, ro.T), generator=g, device="cuda") < p_skip).to(torch.uint8)
    fil = torch.empty_like(i["values"])
    ws = B.Workspace(ro.N, ro.T)
    call = lambda: B.rlcs_gae_skip(i["rewards"], i["values"], i["dones"], i["truncs"], i["trunc_bootstrap"],
                                   i["bootstrap"], skip=skip, gamma=p["gamma"], lam=p["lam"], values_filled=fil,
                                   advantages=o["gae"][0], returns=o["gae"][1], workspace=ws)
    for _ in range(3):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ab = algorithmic_bytes(ro, "gae") + 5 * ro.N * ro.T
    gbs = ab / (ms * 1e-3) / 1e9
    return {"ms": round(ms, 5), "launches_per_call": 1, "p_skip": p_skip, "env_steps_per_s": ro.N * ro.T / (ms * 1e-3),
            "algorithmic_bytes": ab, "gbs": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4)}


def time_retrace_probs(torch, B, steps: int, peak: float, N=16384, T=2048, A=4):
    """Extension beyond the seven kernels: Retrace from [N,T,A] Q-values / action probabilities.
    Algorithmic bytes per step: Q and pi rows (8A), one 32-byte sector of mu for the gathered
    probability (min(32, 4A)), reward 4, action 4, two masks 2, output 4."""
    from paper_2608_17641_b200 import workloads
    ro = workloads.make_rollout(5, N, T, salt=1)
    q, pi, mu, act = workloads.make_action_tensors(5, N, T, A)
    up = lambda a: torch.from_numpy(a).cuda()
    r, d, tr, bv, bt = up(ro.rewards), up(ro.dones), up(ro.truncs), up(ro.trunc_bootstrap), up(ro.bootstrap)
    qd, pid, mud, actd = up(q), up(pi), up(mu), up(act)
    out = torch.empty((N, T), dtype=torch.float32, device="cuda")
    ws = B.Workspace(N, T)
    call = lambda: B.rlcs_retrace_probs(r, qd, pid, mud, actd, d, tr, bv, bt, gamma=0.99, lam=0.95, c_bar=1.0,
                                        q_targets=out, workspace=ws)
    for _ in range(3):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ab = N * T * (8 * A + min(32, 4 * A) + 14) + 4 * N
    gbs = ab / (ms * 1e-3) / 1e9
    return {"ms": round(ms, 5), "N": N, "T": T, "A": A, "env_steps_per_s": N * T / (ms * 1e-3), "algorithmic_bytes": ab,
            "gbs": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4)}


def time_elig_trace_vec(torch, B, steps: int, peak: float, N: int, T: int, D: int, per_dim: bool = False):
    """Extension beyond the seven kernels: vector-valued eligibility traces x[N,T,D] -> z[N,T,D], with
    the shared scalar decay or (per_dim) a decay tensor beta[N,T,D] ~ U(0.5, 1).
    Algorithmic bytes: one read of x (and beta), one write of z, the [N,T] flag."""
    g = torch.Generator(device="cuda").manual_seed(17641)
    x = torch.randn((N, T, D), generator=g, device="cuda", dtype=torch.float32)
    d = (torch.rand((N, T), generator=g, device="cuda") < 0.02).to(torch.uint8)
    out = torch.empty_like(x)
    if per_dim:
        beta = torch.rand((N, T, D), generator=g, device="cuda", dtype=torch.float32) * 0.5 + 0.5
        nbytes = int(B.lib().rlcs_elig_trace_vec_beta_workspace_bytes(N, T, D))
        ws = B.Workspace(N, T, nbytes=nbytes) if nbytes else None
        call = lambda: B.rlcs_elig_trace_vec_beta(x, beta, d, traces=out, workspace=ws)
    else:
        nbytes = int(B.lib().rlcs_elig_trace_vec_workspace_bytes(N, T, D))
        ws = B.Workspace(N, T, nbytes=nbytes) if nbytes else None
        call = lambda: B.rlcs_elig_trace_vec(x, d, gamma=0.99, lam=0.95, traces=out, workspace=ws)
    for _ in range(3):
        call()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(steps):
        call()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / steps
    ab = N * T * ((12 if per_dim else 8) * D + 1)
    gbs = ab / (ms * 1e-3) / 1e9
    return {"ms": round(ms, 5), "N": N, "T": T, "D": D, "workspace_bytes": nbytes, "algorithmic_bytes": ab,
            "gbs": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4)}


def time_time_major(torch, B, steps: int, peak: float, N: int, T: int):
    """Extension beyond the row-major API: the seven algorithms on time-major [T, N] tensors (element
    (t, n) at t*N + n), same value distributions as the headline workload.  Algorithmic bytes as in
    algorithmic_bytes(): every input read once, every output written once, and of the truncation
    continuation values only the 32-byte sectors that hold one the kernel must read."""
    g = torch.Generator(device="cuda").manual_seed(17641)
    mk = lambda scale=1.0: torch.randn((T, N), generator=g, device="cuda", dtype=torch.float32) * scale
    r, v, q, eq, lr, x, bv = mk(), mk(), mk(), mk(), mk(0.3), mk(), mk()
    d = (torch.rand((T, N), generator=g, device="cuda") < 0.02).to(torch.uint8)
    tr = (torch.rand((T, N), generator=g, device="cuda") < 0.005).to(torch.uint8)
    bt = torch.randn((N,), generator=g, device="cuda", dtype=torch.float32)
    o1, o2 = torch.empty_like(r), torch.empty_like(r)
    nbytes = int(B.lib().rlcs_time_major_workspace_bytes(N, T))
    ws = B.Workspace(N, T, nbytes=max(nbytes, 256))
    S = N * T
    sectors = int(((tr != 0) & (d == 0)).view(-1, 8).any(dim=1).sum().item())
    back = lambda nin, nout: 4 * S * (nin + nout) + 2 * S + 4 * N + 32 * sectors
    fwd = 4 * S * 2 + S
    calls = {
        "gae": (lambda: B.rlcs_gae_time_major(r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, advantages=o1, returns=o2, workspace=ws), back(2, 2)),
        "vtrace": (lambda: B.rlcs_vtrace_time_major(r, v, lr, d, tr, bv, bt, gamma=0.99, vs=o1, pg_advantages=o2, workspace=ws), back(3, 2)),
        "retrace": (lambda: B.rlcs_retrace_time_major(r, q, eq, lr, d, tr, bv, bt, gamma=0.99, lam=0.95, q_targets=o1, workspace=ws), back(4, 1)),
        "td_lambda": (lambda: B.rlcs_td_lambda_time_major(r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, returns=o1, workspace=ws), back(2, 1)),
        "discounted_return": (lambda: B.rlcs_discounted_return_time_major(r, d, tr, bv, bt, gamma=0.99, returns=o1, workspace=ws), back(1, 1)),
        "elig_trace": (lambda: B.rlcs_elig_trace_time_major(x, d, gamma=0.99, lam=0.95, traces=o1, workspace=ws), fwd),
        "episodic_prefix_sum": (lambda: B.rlcs_episodic_prefix_sum_time_major(x, d, sums=o1, workspace=ws), fwd),
    }
    out = {"N": N, "T": T, "time_axis_cut": bool(nbytes), "per_algorithm": {}}
    tot_ms = tot_b = 0.0
    for name, (call, ab) in calls.items():
        for _ in range(3):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        gbs = ab / (ms * 1e-3) / 1e9
        out["per_algorithm"][name] = {"ms": round(ms, 5), "algorithmic_bytes": ab, "gbs": round(gbs, 1),
                                      "frac_of_peak": round(gbs / peak, 4)}
        tot_ms += ms
        tot_b += ab
    out["ms_per_step"] = round(tot_ms, 5)
    out["env_steps_per_s"] = round(len(calls) * S / (tot_ms * 1e-3), 1)
    out["all_kernels_frac"] = round(tot_b / (tot_ms * 1e-3) / 1e9 / peak, 4)
    return out


def time_bf16(torch, B, steps: int, peak: float, N: int, T: int):
    """Extension beyond the fp32 method: the seven algorithms on bfloat16 tensors (fp32 arithmetic on
    chip).  Algorithmic bytes: 2 per float element read or written, 1 per mask byte, the bootstrap, and
    of the truncation continuation values the 32-byte sectors (16 values) that hold one the kernel needs."""
    g = torch.Generator(device="cuda").manual_seed(17641)
    mk = lambda scale=1.0: (torch.randn((N, T), generator=g, device="cuda", dtype=torch.float32) * scale).to(torch.bfloat16)
    r, v, q, eq, lr, x, bv = mk(), mk(), mk(), mk(), mk(0.3), mk(), mk()
    d = (torch.rand((N, T), generator=g, device="cuda") < 0.02).to(torch.uint8)
    tr = (torch.rand((N, T), generator=g, device="cuda") < 0.005).to(torch.uint8)
    bt = torch.randn((N,), generator=g, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    o1, o2 = torch.empty_like(r), torch.empty_like(r)
    ws = B.Workspace(N, T)
    S = N * T
    sectors = int(((tr != 0) & (d == 0)).view(-1, 16).any(dim=1).sum().item())
    back = lambda nin, nout: 2 * S * (nin + nout) + 2 * S + 2 * N + 32 * sectors
    fwd = 2 * S * 2 + S
    calls = {
        "gae": (lambda: B.rlcs_gae_bf16(r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, advantages=o1, returns=o2, workspace=ws), back(2, 2)),
        "vtrace": (lambda: B.rlcs_vtrace_bf16(r, v, lr, d, tr, bv, bt, gamma=0.99, vs=o1, pg_advantages=o2, workspace=ws), back(3, 2)),
        "retrace": (lambda: B.rlcs_retrace_bf16(r, q, eq, lr, d, tr, bv, bt, gamma=0.99, lam=0.95, q_targets=o1, workspace=ws), back(4, 1)),
        "td_lambda": (lambda: B.rlcs_td_lambda_bf16(r, v, d, tr, bv, bt, gamma=0.99, lam=0.95, returns=o1, workspace=ws), back(2, 1)),
        "discounted_return": (lambda: B.rlcs_discounted_return_bf16(r, d, tr, bv, bt, gamma=0.99, returns=o1, workspace=ws), back(1, 1)),
        "elig_trace": (lambda: B.rlcs_elig_trace_bf16(x, d, gamma=0.99, lam=0.95, traces=o1, workspace=ws), fwd),
        "episodic_prefix_sum": (lambda: B.rlcs_episodic_prefix_sum_bf16(x, d, sums=o1, workspace=ws), fwd),
    }
    out = {"N": N, "T": T, "per_algorithm": {}}
    tot_ms = tot_b = 0.0
    for name, (call, ab) in calls.items():
        for _ in range(3):
            call()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            call()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        gbs = ab / (ms * 1e-3) / 1e9
        out["per_algorithm"][name] = {"ms": round(ms, 5), "algorithmic_bytes": ab, "gbs": round(gbs, 1),
                                      "frac_of_peak": round(gbs / peak, 4)}
        tot_ms += ms
        tot_b += ab
    out["ms_per_step"] = round(tot_ms, 5)
    out["env_steps_per_s"] = round(len(calls) * S / (tot_ms * 1e-3), 1)
    out["all_kernels_frac"] = round(tot_b / (tot_ms * 1e-3) / 1e9 / peak, 4)
    return out


def time_e2e(batch: GpuBatch, steps: int, warmup: int, dist):
    """The same step called with HOST buffers: every step copies that step's inputs from pinned
    host memory to the device, runs the seven C-ABI calls, and reads all outputs back to pinned
    host memory.  Three streams, as a caller would arrange them: copies in, kernels, copies out;
    a kernel starts as soon as its own inputs have landed, and one step's read-back overlaps the
    next step's upload (the link is full duplex).  Inputs and outputs are single-buffered on the
    device, so uploads wait for the previous step's kernels and kernels for the previous read-back."""
    torch, ro = batch.torch, batch.ro
    pin = lambda t: torch.empty(t.shape, dtype=t.dtype).pin_memory().copy_(t.cpu())
    h_in = {k: pin(v) for k, v in batch.inp.items() if v is not None}
    h_out = {}
    for a, v in batch.out.items():
        h_out[a] = tuple(torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in v) if isinstance(v, tuple) \
            else torch.empty(v.shape, dtype=v.dtype).pin_memory()
    h2d = sum(t.numel() * t.element_size() for t in h_in.values())
    d2h = sum(t.numel() * t.element_size() for v in h_out.values() for t in (v if isinstance(v, tuple) else (v,)))
    s_in, s_k, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    # upload order and the algorithms that can start after each group
    groups = [(("dones", "truncs", "bootstrap", "trunc_bootstrap", "rewards", "values"), ("gae", "td_lambda", "discounted_return")),
              (("log_rhos",), ("vtrace",)), (("q_sa", "expected_q"), ("retrace",)),
              (("x", "any_done"), ("elig_trace", "episodic_prefix_sum"))]
    state = {"kernels_done": None, "readback_done": None}

    def one():
        if state["kernels_done"] is not None:
            s_in.wait_event(state["kernels_done"])          # the previous step still reads the inputs
        if state["readback_done"] is not None:
            s_k.wait_event(state["readback_done"])          # ... and its outputs are still being read back
        for names, algos in groups:
            with torch.cuda.stream(s_in):
                for k in names:
                    if k in h_in:
                        batch.inp[k].copy_(h_in[k], non_blocking=True)
                landed = torch.cuda.Event()
                landed.record(s_in)
            s_k.wait_event(landed)
            for a in algos:
                with torch.cuda.stream(s_k):
                    batch.call(a)
                    ran = torch.cuda.Event()
                    ran.record(s_k)
                s_out.wait_event(ran)
                with torch.cuda.stream(s_out):
                    v = batch.out[a]
                    for hv, dv in zip(h_out[a] if isinstance(v, tuple) else (h_out[a],), v if isinstance(v, tuple) else (v,)):
                        hv.copy_(dv, non_blocking=True)
        state["kernels_done"] = torch.cuda.Event()
        state["kernels_done"].record(s_k)
        state["readback_done"] = torch.cuda.Event()
        state["readback_done"].record(s_out)

    cur = torch.cuda.current_stream()
    for s in (s_in, s_k, s_out):
        s.wait_stream(cur)
    for _ in range(warmup):
        one()
    for s in (s_in, s_k, s_out):
        cur.wait_stream(s)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist.barrier()
    torch.cuda.synchronize()
    start.record(cur)
    for s in (s_in, s_k, s_out):
        s.wait_stream(cur)
    for _ in range(steps):
        one()
    for s in (s_in, s_k, s_out):
        cur.wait_stream(s)
    stop.record(cur)
    torch.cuda.synchronize()
    dist.barrier()
    return start.elapsed_time(stop), h2d, d2h


# --------------------------------------------------------------------------------------------- CPU oracle arm
def oracle_pass(ro, rows: int, threads: int):
    """All seven algorithms of the oracle, as it stands, on the first `rows` rows; returns seconds."""
    import oracle
    p = ro.params
    s = slice(0, rows)
    cut = lambda a: None if a is None else a[s]
    bw2 = dict(dones=cut(ro.dones), truncs=cut(ro.truncs), trunc_bootstrap=cut(ro.trunc_bootstrap))
    bw1 = dict(bootstrap=cut(ro.bootstrap))
    d_fwd = cut(ro.any_done)
    par = lambda fn, a2, a1, **kw: oracle.run_rows_parallel(fn, a2, a1, threads, **kw)
    t0 = time.perf_counter()
    par(oracle.gae, dict(rewards=cut(ro.rewards), values=cut(ro.values), **bw2), bw1, gamma=p["gamma"], lam=p["lam"])
    par(oracle.vtrace, dict(rewards=cut(ro.rewards), values=cut(ro.values), log_rhos=cut(ro.log_rhos), **bw2), bw1,
        gamma=p["gamma"], rho_bar=p["rho_bar"], c_bar=p["c_bar"])
    par(oracle.retrace, dict(rewards=cut(ro.rewards), q_sa=cut(ro.q_sa), expected_q=cut(ro.expected_q),
                             log_rhos=cut(ro.log_rhos), **bw2), bw1, gamma=p["gamma"], lam=p["lam"], c_bar=p["c_bar"])
    par(oracle.td_lambda, dict(rewards=cut(ro.rewards), values=cut(ro.values), **bw2), bw1, gamma=p["gamma"], lam=p["lam"])
    par(oracle.discounted_return, dict(rewards=cut(ro.rewards), **bw2), bw1, gamma=p["gamma"])
    par(oracle.elig_trace, dict(x=cut(ro.x), dones=d_fwd), {}, gamma=p["gamma"], lam=p["lam"])
    par(oracle.episodic_prefix_sum, dict(x=cut(ro.x), dones=d_fwd), {})
    return time.perf_counter() - t0


def cpu_baseline(ro, budget_s: float = 20.0):
    import oracle
    oracle.build()
    threads = os.cpu_count() or 1
    probe_rows = min(ro.N, 256)
    t = oracle_pass(ro, probe_rows, threads)                          # calibration (also warms the library)
    rows = int(min(ro.N, max(probe_rows, probe_rows * budget_s / max(t, 1e-6))))
    secs = oracle_pass(ro, rows, threads)
    rows1 = int(min(rows, max(64, rows * 3.0 / max(secs * threads, 1e-3))))   # about 3 CPU-seconds' worth of rows at the multi-thread rate
    secs1 = oracle_pass(ro, rows1, 1)
    return {"value": len(ALGOS) * rows * ro.T / secs, "unit": METRIC, "cores": threads, "kind": "oracle",
            "single_thread_value": len(ALGOS) * rows1 * ro.T / secs1, "cpu_model": _cpu_model(),
            "sample": f"first {rows} of {ro.N} rows x T={ro.T}, all seven algorithms once, {secs:.2f} s, "
                      f"fp64 sequential C oracle, rows split over {threads} host threads "
                      f"(single thread: first {rows1} rows, {secs1:.2f} s)"}


def _cpu_model() -> str:
    try:
        with open("/proc/cpuinfo") as fh:
            for line in fh:
                if line.lower().startswith("model name"):
                    return line.split(":", 1)[1].strip()
    except OSError:
        pass
    return "unknown"


def reference_arm(args, world: int):
    """The CPU oracle on the bench workload; each step is a bounded row sample of it."""
    from paper_2608_17641_b200 import workloads
    import oracle
    oracle.build()
    ro = workloads.config5(**WORKLOAD)
    threads = os.cpu_count() or 1
    probe = 128
    t = oracle_pass(ro, probe, threads)
    per_step_budget = 150.0 / max(1, args.steps + args.warmup)
    rows = int(min(ro.N, max(16, probe * per_step_budget / max(t, 1e-6))))
    for _ in range(args.warmup):
        oracle_pass(ro, rows, threads)
    times = [oracle_pass(ro, rows, threads) for _ in range(args.steps)]
    total = sum(times)
    value = len(ALGOS) * rows * ro.T * args.steps / total
    sample = (f"each step = first {rows} of {ro.N} rows x T={ro.T}, all seven algorithms, fp64 sequential C oracle, "
              f"rows split over {threads} host threads")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": METRIC, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"all seven algorithms, num_envs={ro.N}, T={ro.T}, fp32 inputs, truncation handling on "
                               f"(bounded row sample per step)", "rows_per_step": rows},
        "cpu_baseline": {"value": value, "unit": METRIC, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": METRIC, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------- sweeps (cold L2)
def sweep_case(torch, B, ro, algo: str, use_truncs: bool, hbm_peak: float, l2_bytes: int, trials=5, ceilings=True):
    """Device time per call with a cold L2: the calls of one batch rotate over R distinct copies of
    all inputs and outputs whose total footprint exceeds 3x the L2 capacity."""
    ro_eff = ro if use_truncs else _without_truncs(ro)
    algo_bytes = algorithmic_bytes(ro_eff, algo)
    R = int(min(512, max(4, -(-3 * l2_bytes // algo_bytes))))
    sets = [GpuBatch(ro_eff, torch.device("cuda", torch.cuda.current_device()), only=algo) for _ in range(R)]
    call = lambda i: sets[i].call(algo)
    for i in range(R):
        call(i)
    torch.cuda.synchronize()
    # device time: the R launches replayed from a CUDA graph (no host launch cost between kernels)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(R):
            call(i)
    graph.replay()
    per_call_us, full_call_us = [], []
    for _ in range(trials):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        per_call_us.append(1e3 * e0.elapsed_time(e1) / R)
    # full call: the same launches issued one by one through the Python binding
    for _ in range(trials):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for i in range(R):
            call(i)
        e1.record()
        torch.cuda.synchronize()
        full_call_us.append(1e3 * e0.elapsed_time(e1) / R)
    # ... and through prepared calls (arguments marshalled once, then only the C call)
    prepared_us = []
    if ceilings:
        steps = [b.prepared(algo) for b in sets]
        h = torch.cuda.current_stream().cuda_stream
        for _ in range(trials):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            e0.record()
            for st in steps:
                st(h)
            e1.record()
            torch.cuda.synchronize()
            prepared_us.append(1e3 * e0.elapsed_time(e1) / R)
        del steps
    best = min(per_call_us)
    gbs = algo_bytes / (best * 1e-6) / 1e9
    del sets, graph
    if not ceilings:
        return {"algo": algo, "N": ro.N, "T": ro.T, "truncs": use_truncs, "us_per_call": round(best, 3),
                "us_per_call_median": round(statistics.median(per_call_us), 3), "algorithmic_bytes": algo_bytes,
                "gbs": round(gbs, 1), "frac_of_peak": round(gbs / hbm_peak, 4), "rotating_sets": R,
                "timing": "CUDA-graph replay of launches rotating over buffer sets > 3x L2"}
    ceiling_us = copy_ceiling_us(torch, B, ro_eff, algo, algo_bytes, R, trials)
    ceiling_gbs = algo_bytes / (ceiling_us * 1e-6) / 1e9
    memcpy_us = memcpy_ceiling_us(torch, algo_bytes, R, trials)
    return {"algo": algo, "N": ro.N, "T": ro.T, "truncs": use_truncs, "us_per_call": round(best, 3),
            "copy_ceiling_us": round(ceiling_us, 3), "copy_ceiling_gbs": round(ceiling_gbs, 1),
            "memcpy_ceiling_us": round(memcpy_us, 3), "frac_of_memcpy_ceiling": round(memcpy_us / best, 4),
            "frac_of_copy_ceiling": round(gbs / ceiling_gbs, 4),
            "us_per_call_median": round(statistics.median(per_call_us), 3),
            "full_call_us": round(min(full_call_us), 3), "prepared_call_us": round(min(prepared_us), 3), "env_steps_per_s": ro.N * ro.T / (best * 1e-6),
            "algorithmic_bytes": algo_bytes, "gbs": round(gbs, 1), "frac_of_peak": round(gbs / hbm_peak, 4),
            "rotating_sets": R, "l2": "cold (rotating buffer sets > 3x L2)", "timing": "CUDA-graph replay of the rotating launches"}


def copy_ceiling_us(torch, B, ro, algo: str, algo_bytes: int, R: int, trials: int) -> float:
    """Device time of a plain streaming kernel at the same byte count, read:write ratio and cold-L2
    rotation as one scan launch of this case: what the size itself allows."""
    S = ro.N * ro.T
    write_bytes = 4 * S * {"gae": 2, "vtrace": 2}.get(algo, 1)
    read_bytes = max(32, algo_bytes - write_bytes)
    rd = [torch.empty(read_bytes // 4 + 8, dtype=torch.float32, device="cuda").normal_() for _ in range(R)]
    wr = [torch.empty(write_bytes // 4 + 8, dtype=torch.float32, device="cuda") for _ in range(R)]
    call = lambda i: B.rlcs_debug_stream_copy(rd[i], wr[i], read_bytes, write_bytes)
    for i in range(R):
        call(i)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(R):
            call(i)
    graph.replay()
    times = []
    for _ in range(trials):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(1e3 * e0.elapsed_time(e1) / R)
    return min(times)


def memcpy_ceiling_us(torch, algo_bytes: int, R: int, trials: int) -> float:
    """A second, independent ceiling: the driver's own device-to-device copy (cudaMemcpyAsync through
    torch's copy_) moving the same total of bytes -- half of them read, half written -- in the same
    cold-L2 rotation and CUDA-graph replay as the scan launches."""
    n = -(-(algo_bytes // 2 // 4) // 4096) * 4096          # whole 16 KB pieces: odd sizes take a slower copy path
    rd = [torch.empty(n, dtype=torch.float32, device="cuda").normal_() for _ in range(R)]
    wr = [torch.empty(n, dtype=torch.float32, device="cuda") for _ in range(R)]
    for i in range(R):
        wr[i].copy_(rd[i])
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for i in range(R):
            wr[i].copy_(rd[i])
    graph.replay()
    times = []
    for _ in range(trials):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        graph.replay()
        e1.record()
        torch.cuda.synchronize()
        times.append(1e3 * e0.elapsed_time(e1) / R)
    return min(times)


def _without_truncs(ro):
    import copy
    r2 = copy.copy(ro)
    r2.truncs = None
    r2.trunc_bootstrap = None
    return r2


def small_config_summary(sweeps) -> dict:
    """frac_of_peak of the cold-L2 cases the bandwidth target names: N=4096 with T >= 256, and the
    long-row configuration (64 x 16384).  Keys: <algo>_<T>[t]; t = with truncation handling."""
    short = {"gae": "gae", "vtrace": "vtr", "discounted_return": "disc"}
    out = {}
    for c in sweeps:
        if (c["N"] == 4096 and c["T"] >= 256) or c["T"] == 16384:
            out[f"{short.get(c['algo'], c['algo'])}_{c['T']}{'t' if c['truncs'] else ''}"] = round(c["frac_of_peak"], 3)
    return out


def run_sweeps(torch, hbm_peak, pick=None, trials=5):
    """The cold-L2 cases of configurations 1-4.  `pick` = (config, algo, T, truncs), None entries
    matching anything, keeps only the matching cases (for a profiler run on one kernel)."""
    from paper_2608_17641_b200 import binding as B, workloads
    l2 = torch.cuda.get_device_properties(0).L2_cache_size
    cases = [(1, lambda: workloads.config1(), "gae", True)]                                    # config 1: latency floor
    cases += [(2, lambda: workloads.config2(), algo, True) for algo in ALGOS]                  # config 2: all seven
    for T in (32, 64, 128, 256, 512, 1024):
        for tr in (False, True):
            cases += [(3, (lambda T=T: workloads.config3(T, True)), algo, tr) for algo in ("gae", "vtrace")]
    cases += [(4, lambda: workloads.config4(), algo, False) for algo in ("gae", "discounted_return")]
    out = []
    for cfg, make, algo, tr in cases:
        if pick is not None and any(want is not None and want != got for want, got in zip(pick[:2], (cfg, algo))):
            continue
        ro = make()
        if pick is not None and ((pick[2] is not None and pick[2] != ro.T) or (pick[3] is not None and pick[3] != tr)):
            continue
        out.append(sweep_case(torch, B, ro, algo, tr, hbm_peak, l2, trials=trials))
    return out


# --------------------------------------------------------------------------------------------- main
class _NoDist:
    rank, world = 0, 1

    def barrier(self):
        pass

    def max(self, x: float) -> float:
        return x

    def sum(self, x: float) -> float:
        return x


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", choices=("ours", "reference"), default="ours")
    ap.add_argument("--no-sweep", action="store_true", help="skip the cold-L2 sweeps of the smaller configurations")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--sweep-only", action="store_true", help="print only the cold-L2 sweeps (one JSON line)")
    ap.add_argument("--sweep-pick", default=None, metavar="CONFIG,ALGO,T,TRUNCS",
                    help="with --sweep-only: keep the matching cases only, e.g. 3,vtrace,256,1 or 4,gae,, (empty = any)")
    ap.add_argument("--sweep-trials", type=int, default=5)
    ap.add_argument("--sweep-shape", default=None, metavar="N,T,ALGO,TRUNCS[,P_TRUNC]",
                    help="with --sweep-only: one cold-L2 case on a dense-reward batch of this shape instead of the configurations")
    ap.add_argument("--variant", type=int, default=None, help="tile variant test hook (default: library default)")
    ap.add_argument("--no-dependent-launch", action="store_true",
                    help="measurement hook: launch the scan kernels without programmatic stream serialisation")
    ap.add_argument("--row-blocks", type=int, default=None, help="measurement hook: one thread block per row (0 never, 1 whenever legal)")
    ap.add_argument("--no-row-tiles", action="store_true", help="measurement hook: no row-aligned tiling (short rows use the look-back)")
    ap.add_argument("--no-truncs", action="store_true", help="bench batch without per-step truncation handling")
    ap.add_argument("--rows", type=int, default=WORKLOAD["N"], help="num_envs of the bench batch (default: full size)")
    ap.add_argument("--only", choices=("time_major", "bf16", "retrace_probs", "elig_trace_vec", "elig_trace_vec_beta",
                                       "gae_skip", "gae_normalized"), default=None,
                    help="time only that extension line on a --rows x --seq-len batch and print it (one JSON line)")
    ap.add_argument("--seq-len", type=int, default=WORKLOAD["T"], help="T of the --only batch")
    ap.add_argument("--tm-path", type=int, default=0, help="time-major path test hook for --only runs (0 = library default)")
    ap.add_argument("--detail-file", default=None, help="also write headline + detail lines to this JSON file")
    ap.add_argument("--traffic-from-ncu", default=None, metavar="CSV",
                    help="no benchmark: turn ncu's CSV log of the DRAM byte counters into profiles/dram_traffic_16384x2048.json")
    ap.add_argument("--traffic-command", default="", help="with --traffic-from-ncu: the ncu command line, recorded in the file")
    ap.add_argument("--dim", type=int, default=64, help="D of the --only elig_trace_vec* batch, A of retrace_probs")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.traffic_from_ncu is not None:
        print(json.dumps(traffic_from_ncu(args.traffic_from_ncu, command=args.traffic_command)))
        return

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if args.gpus > 1 and world == 1:
        # not under torchrun: relaunch one rank per GPU
        os.execvp(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                   f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1", "--master-port",
                                   os.environ.get("MASTER_PORT", "29517"), os.path.abspath(__file__), *sys.argv[1:]])

    if args.impl == "reference":
        if rank == 0:
            reference_arm(args, world)
        return

    import torch
    from paper_2608_17641_b200 import binding, workloads
    from paper_2608_17641_b200.distributed import Dist
    binding.lib()                                   # no library, no benchmark: there is no fallback
    if args.variant is not None:
        binding.rlcs_debug_set_tile_variant(args.variant)
    if args.no_dependent_launch:
        binding.rlcs_debug_set_dependent_launch(False)
    if args.no_row_tiles:
        binding.rlcs_debug_allow_row_tiles(False)
    if args.row_blocks is not None:
        binding.rlcs_debug_set_row_blocks(args.row_blocks)
    assert torch.cuda.is_available(), "bench.py needs a CUDA device"
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dist = Dist.from_env(backend="nccl", device=torch.device("cuda", local)) if world > 1 else _NoDist()

    if args.sweep_only:
        peak, _ = measured_peak()
        if args.sweep_shape is not None:
            n, t, a, tr, *rest = args.sweep_shape.split(",")
            ro = workloads.make_rollout(3, int(n), int(t), with_truncs=True, p_trunc=float(rest[0]) if rest else 0.005)
            case = sweep_case(torch, binding, ro, a, bool(int(tr)), peak, torch.cuda.get_device_properties(0).L2_cache_size,
                              trials=max(1, args.sweep_trials))
            print(json.dumps({"detail": "sweep", **case}), flush=True)
            return
        pick = None
        if args.sweep_pick is not None:
            c, a, t, tr = (args.sweep_pick.split(",") + ["", "", "", ""])[:4]
            pick = (int(c) if c else None, a or None, int(t) if t else None, bool(int(tr)) if tr else None)
        for case in run_sweeps(torch, peak, pick, max(1, args.sweep_trials)):
            print(json.dumps({"detail": "sweep", **case}), flush=True)
        return
    if args.only is not None:
        peak, _ = measured_peak()
        binding.rlcs_debug_time_major_path(args.tm_path)
        k, N, T = max(1, args.steps), args.rows, args.seq_len
        if args.only in ("time_major", "bf16"):
            res = (time_time_major if args.only == "time_major" else time_bf16)(torch, binding, k, peak, N, T)
        elif args.only == "retrace_probs":
            res = time_retrace_probs(torch, binding, k, peak, N, T, args.dim)
        elif args.only in ("elig_trace_vec", "elig_trace_vec_beta"):
            res = time_elig_trace_vec(torch, binding, k, peak, N, T, args.dim, per_dim=args.only.endswith("beta"))
        else:
            batch = GpuBatch(workloads.config5(N=N, T=T, salt=rank), torch.device("cuda", local))
            res = (time_gae_skip if args.only == "gae_skip" else time_gae_normalized)(batch, k, peak)
        print(json.dumps({args.only: res}), flush=True)
        return

    N = args.rows
    ro = workloads.config5(N=N, T=WORKLOAD["T"], salt=rank)        # every rank draws its own batch
    if args.no_truncs:
        ro.truncs = None
        ro.trunc_bootstrap = None
    batch = GpuBatch(ro, torch.device("cuda", local))
    total_ms, per_algo_ms, launches, clocks = time_device(batch, args.steps, args.warmup, dist)
    total_ms = dist.max(total_ms)
    units_per_step = len(ALGOS) * ro.N * ro.T * world
    value = units_per_step * args.steps / (total_ms * 1e-3)

    peak, peak_kind = measured_peak()
    per_algo = {}
    for a in ALGOS:
        ms = statistics.median(per_algo_ms[a])
        ab = algorithmic_bytes(ro, a)
        gbs = ab / (ms * 1e-3) / 1e9
        per_algo[a] = {"ms": round(ms, 5), "samples_ms": [round(x, 4) for x in per_algo_ms[a]],
                       "env_steps_per_s": ro.N * ro.T / (ms * 1e-3), "algorithmic_bytes": ab,
                       "gbs": round(gbs, 1), "frac_of_peak": round(gbs / peak, 4)}
        if ro.truncs is not None and a not in ("elig_trace", "episodic_prefix_sum"):
            # the same time against the byte count of a kernel that would read trunc_bootstrap densely (context only)
            dense = 4 * ro.N * ro.T * ({"gae": 4, "vtrace": 5, "retrace": 5, "td_lambda": 3, "discounted_return": 2}[a] + 1) \
                + 2 * ro.N * ro.T + 4 * ro.N
            per_algo[a]["gbs_dense_trunc_bootstrap_count"] = round(dense / (ms * 1e-3) / 1e9, 1)
    dom = max(ALGOS, key=lambda a: per_algo[a]["ms"])
    full_size = (ro.N, ro.T) == (WORKLOAD["N"], WORKLOAD["T"]) and ro.truncs is not None
    traffic_table = load_traffic() if full_size else {}
    for a in ALGOS:
        per_algo[a]["kernel"] = kernel_instance(binding, a, ro.truncs is not None, ro.N, ro.T)
        per_algo[a]["ncu_dram_bytes"] = traffic_for(a, per_algo[a]["kernel"], traffic_table)
    roofline = {"bound": "hbm", "kernel": f"{per_algo[dom]['kernel']} ({dom})",
                "achieved": per_algo[dom]["gbs"], "peak": peak, "unit": "GB/s",
                "frac": round(per_algo[dom]["gbs"] / peak, 4), "traffic": per_algo[dom]["ncu_dram_bytes"],
                "algorithmic_bytes_per_launch": per_algo[dom]["algorithmic_bytes"], "peak_source": f"of {peak_kind}",
                "all_kernels_frac": round(sum(v["algorithmic_bytes"] for v in per_algo.values())
                                          / (sum(v["ms"] for v in per_algo.values()) * 1e-3) / 1e9 / peak, 4)}
    details = [{"detail": "per_algorithm", "N": ro.N, "T": ro.T, "truncs": ro.truncs is not None, "per_algorithm": per_algo}]

    ext = lambda name, res: details.append({"detail": "extension", "name": name, "result": res})
    ext("gae_normalized", time_gae_normalized(batch, max(3, min(args.steps, 50)), peak))
    if rank == 0 and world == 1 and not args.no_sweep:
        ext("gae_skip", time_gae_skip(batch, max(3, min(args.steps, 30)), peak))
    e2e_steps = max(1, min(args.steps, 8))
    e2e_ms, h2d, d2h = time_e2e(batch, e2e_steps, 1, dist)
    e2e_ms = dist.max(e2e_ms)
    e2e = {"value": units_per_step * e2e_steps / (e2e_ms * 1e-3), "unit": METRIC, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": round(e2e_ms / e2e_steps, 4),
           "note": "pinned host -> device, seven C-ABI calls, all outputs -> pinned host; three streams"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(ro)
        details.append({"detail": "cpu_baseline", **cpu})
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample")}
    small = None
    if rank == 0 and world == 1 and not args.no_sweep:
        del batch
        torch.cuda.empty_cache()
        k30, k20 = max(3, min(args.steps, 30)), max(3, min(args.steps, 20))
        # the same number of steps as the bench batch in long rows (token-level trajectories): the two
        # GAE extensions on rows of 8192 steps
        long_rows = GpuBatch(workloads.config5(N=WORKLOAD["N"] // 4, T=WORKLOAD["T"] * 4, salt=rank), torch.device("cuda", local))
        ext("gae_skip_long_rows", {"N": long_rows.ro.N, "T": long_rows.ro.T, **time_gae_skip(long_rows, k20, peak)})
        ext("gae_normalized_long_rows", {"N": long_rows.ro.N, "T": long_rows.ro.T, **time_gae_normalized(long_rows, k20, peak)})
        del long_rows
        torch.cuda.empty_cache()
        ext("retrace_probs", time_retrace_probs(torch, binding, k30, peak))
        ext("elig_trace_vec", [time_elig_trace_vec(torch, binding, k30, peak, *shape)
                               for shape in ((4096, 512, 64), (1024, 1024, 64), (64, 16384, 64), (16, 65536, 64))])
        ext("elig_trace_vec_beta", [time_elig_trace_vec(torch, binding, k30, peak, *shape, per_dim=True)
                                    for shape in ((16384, 128, 64), (4096, 512, 64), (64, 16384, 64), (16, 65536, 64))])
        for shape in ((WORKLOAD["N"], WORKLOAD["T"]), (65536, 512), (2048, 2048)):
            ext("time_major", time_time_major(torch, binding, k20, peak, *shape))
        torch.cuda.empty_cache()
        ext("bf16", time_bf16(torch, binding, k20, peak, WORKLOAD["N"], WORKLOAD["T"]))
        torch.cuda.empty_cache()
        # the seven kernels of the headline workload launched back to back (no event between launches):
        # what each sustains when its ramp-up and tail overlap its neighbours', as they do in a step
        l2 = torch.cuda.get_device_properties(0).L2_cache_size
        details += [{"detail": "back_to_back", **sweep_case(torch, binding, ro, a, ro.truncs is not None, peak, l2, trials=3, ceilings=False)}
                    for a in ALGOS]
        torch.cuda.empty_cache()
        sweeps = run_sweeps(torch, peak)
        details += [{"detail": "sweep", **c} for c in sweeps]
        small = small_config_summary(sweeps)
    if rank == 0:
        workload = (f"config 5: all seven algorithms, num_envs={ro.N}, T={ro.T}, fp32, dones~Bern(0.02), truncs~Bern(0.005) "
                    f"with per-step truncation handling, gamma=0.99, lambda=0.95; {len(ALGOS)} launches per step")
        headline = build_headline(value=value, world=world, steps=args.steps, warmup=args.warmup,
                                  ms_per_step=round(total_ms / args.steps, 5), workload=workload, clocks=clocks, e2e=e2e,
                                  launches=launches, roofline=roofline, cpu_baseline=cpu,
                                  per_algorithm_frac={a: per_algo[a]["frac_of_peak"] for a in ALGOS}, small_frac=small,
                                  detail_file=args.detail_file)
        emit(details, headline, args.detail_file)
    if world > 1:
        dist.close()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the windowed-attention hot path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--workload NAME]

One step = one pass of the whole hot path over one batch of seeded synthetic input:
window table (host) -> RoPE of Q and K -> windowed causal prefill, which also writes the tiled
group-major K cache -> one windowed decode step on the cache just written (no conversion in
between).  The default workload is the Llama-3.2-3B attention-layer shape at 128K tokens (the
configuration the headline metric is quoted on).  Prints ONE JSON line.

With --gpus N every rank runs an independent replica (the path has no exchange step); rank 0 reports
the aggregate with the max-over-ranks time.  Under torchrun the ranks are the launcher's; a plain
`python bench.py --gpus N` (N > 1) starts the N ranks itself.
"""
from __future__ import annotations

import argparse
import datetime
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

import atf_inputs as gen  # noqa: E402

METRIC = "prefill executed TFLOP/s at 128K (with ms, decode us/step and HBM GB/s alongside)"
T = 128  # tile edge of the prefill kernel (query rows and keys per tile)


def workload_by_name(name):
    if name == "llama3b-128k":
        return gen.llama32_3b(131072, B=1, seed_off=6)
    if name == "llama3b-32k":
        return gen.llama32_3b(32768, B=1, seed_off=5)
    if name == "llama3b-8k":
        return gen.llama32_3b(8192, B=1, seed_off=4)
    if name == "llama3b-128k-b8":   # decode only: eight sequences
        return gen.llama32_3b(131072, B=8, seed_off=10)
    if name == "llama3b-32k-b8":
        return gen.llama32_3b(32768, B=8, seed_off=8)
    if name == "qwen05b-8k":
        return gen.qwen05b(8192)
    if name == "qwen05b-32k":
        return gen.qwen05b(32768)
    if name == "qwen7b-1m":
        return gen.qwen7b_1m(1 << 20)
    if name == "tiny":
        return gen.tiny()
    raise SystemExit(f"unknown workload {name}")


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops"],
                "bf16_tflops_sustained": j.get("bf16_tflops_sustained", j["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# ---- work accounting (definitions only: Sec. 4's term count turned into FLOPs and bytes) ----
def kept_terms_prefill(W, N):
    tot = 0
    for w in W:
        w = int(w)
        a = min(w, N - 1)
        tot += (a + 1) * (a + 2) // 2 + max(0, N - 1 - w) * (w + 1)
    return tot


def kept_terms_decode(W, L):
    return sum(min(int(w), L - 1) + 1 for w in W)


def prefill_flops(wl, W, n0=0):
    """Executed and effective FLOPs of the query rows n0..N-1 (n0 = 0: the whole prefill)."""
    cells = wl.N * (wl.N + 1) // 2 - n0 * (n0 + 1) // 2
    kept = kept_terms_prefill(W, wl.N) - (kept_terms_prefill(W, n0) if n0 else 0)
    executed = wl.B * wl.Hq * (4 * kept + 2 * wl.d * cells)
    effective = wl.B * wl.Hq * 4 * wl.d * cells
    return executed, effective


def prefill_issued_flops(wl, W, coarse=False):
    """FLOPs of the tensor-core products the prefill kernel actually launches: per (128-row query tile, 128-key
    tile) at tile distance dt a 128 x 128 x 16 product per 16-column step of the tile's depth (the band schedule:
    exact mode keeps the pairs live at the distance from the middle of the nearest row quarter to the middle of the
    tile, coarse mode the pairs live anywhere in the tile, both rounded up to 8 pairs; the diagonal tile runs at
    full depth in coarse mode), plus the 128 x d x 128 product P V.  Padding of the last tiles, the masked half of
    the diagonal tiles and pairs kept in the product although dead in some cells are all in; tile distances no
    pair reaches are not launched."""
    h = wl.d // 2
    W = [int(w) for w in W]
    nt = (wl.N + T - 1) // T
    dlim = (W[-1] + T - 1) // T + 1

    def reaching(z):  # pairs with w >= z
        return sum(1 for w in W if w >= z)
    total = 0
    for dt in range(min(nt, dlim)):
        if coarse:
            depth = h if dt == 0 else min(h, (reaching(dt * T - (T - 1)) + 7) // 8 * 8)
        else:
            depth = reaching(15 if dt == 0 else dt * T - 48)
        natoms = (depth + 7) // 8
        tiles = nt - dt
        total += tiles * (natoms * 2 * T * T * 16 + (T // 16) * 2 * T * wl.d * 16)
    return wl.B * wl.Hq * total


def decode_bytes(wl, W, windowed=True):
    L = wl.N
    kept = kept_terms_decode(W, L) if windowed else (wl.d // 2) * L
    return wl.B * wl.Hkv * (4 * kept + 2 * wl.d * L)


def decode_fetched_bytes(wl, W):
    """Bytes the group-major decode asks for: per tile of KT keys the groups of 8 pairs its nearest key keeps
    (32 bytes per key and group), plus V in full."""
    L, h = wl.N, wl.d // 2
    kt = 8192 // wl.d
    W = [int(w) for w in W]
    tot = 0
    for t in range((L + kt - 1) // kt):
        z_near = max(L - 1 - (t * kt + kt - 1), 0)
        live = sum(1 for w in W if w >= z_near)
        if live:
            tot += ((live + 7) // 8) * kt * 32 + kt * wl.d * 2
    return wl.B * wl.Hkv * tot


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons (with time stamps) while the timed regions run."""
    Q = ("timestamp,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index, period_ms=50):
        self.index, self.period_ms = index, period_ms
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-i", str(self.index), "-lms", str(self.period_ms)],
                                         stdout=subprocess.PIPE, text=True)
            self.th = threading.Thread(target=self._read, daemon=True)
            self.th.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            c = [x.strip() for x in line.split(",")]
            try:
                ts = datetime.datetime.strptime(c[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((ts, float(c[1]), float(c[2]), c[4:8]))
            except Exception:
                continue

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                self.proc.kill()

    def summary(self, t0=None, t1=None):
        """Median SM clock and the throttle reasons seen between two wall-clock times (all samples if None)."""
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"], "samples": 0}
        rows = [r for r in self.rows if (t0 is None or r[0] >= t0) and (t1 is None or r[0] <= t1)]
        reasons = set()
        for r in rows:
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        sm = [r[1] for r in rows if r[1] > 0]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": rows[-1][2] if rows else None,
                "reasons": sorted(reasons), "samples": len(sm)}

    def mhz_in(self, windows):
        """Median SM clock over the samples that fall into any of the (t0, t1) wall-clock windows."""
        sm = [r[1] for r in self.rows if r[1] > 0 and any(a <= r[0] <= b for a, b in windows)]
        return statistics.median(sm) if sm else None


def ev():
    return torch.cuda.Event(enable_timing=True)


def max_over_ranks(ms, device):
    """Replicas share nothing but the clock: the job's time is the slowest rank's."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(per_replica_work, world, ms):
    """Whole-job throughput in T(units)/s: every replica does the same work in the max time."""
    return world * per_replica_work / (ms * 1e-3) / 1e12


def spread(vals):
    return {"median": statistics.median(vals), "min": min(vals), "max": max(vals), "n": len(vals)}


def run_ours(args):
    import paper_2608_02947_b200 as atf

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    atf.lib()  # fails loudly if the CUDA library is missing

    wl = workload_by_name(args.workload)
    pk = peaks()
    if args.decode_only:
        return run_decode_only(args, atf, wl, pk, dev)
    if args.split_precision:
        return run_split_precision(args, atf, wl, dev)
    Q0, K0, V = gen.prefill_inputs(wl, device=dev)  # un-rotated, on the device
    Qg, Kg = Q0.clone(), K0.clone()
    O = torch.empty_like(Qg)
    LSE = torch.empty((wl.B, wl.Hq, wl.N), dtype=torch.float32, device=dev)
    qd = torch.empty((wl.B, wl.Hq, wl.d), dtype=torch.bfloat16, device=dev)
    Od = torch.empty_like(qd)
    Kcache = atf.new_kcache_groups(wl.B, wl.Hkv, wl.N, wl.d, dev)  # written by the prefill, read by the decode
    nbytes = max(atf.atf_workspace_bytes(0, wl.B, wl.Hq, wl.Hkv, wl.N, wl.d),
                 atf.atf_workspace_bytes(1, wl.B, wl.Hq, wl.Hkv, wl.N, wl.d))
    atf.ensure_workspace(nbytes, dev)

    t_rope, t_pre, t_dec = [], [], []

    def step(timed):
        e = [ev() for _ in range(5)]
        e[0].record()
        W, theta = atf.atf_window_table(wl.base, wl.d, wl.k, wl.N, wl.scaling)
        W = atf.WindowTable(W)
        Qg.copy_(Q0)
        Kg.copy_(K0)
        e[1].record()
        atf.atf_rope(Qg, theta)
        atf.atf_rope(Kg, theta)
        e[2].record()
        Wuse = None if args.full_attention else W
        atf.atf_prefill(Qg, Kg, V, table=Wuse, O=O, LSE=LSE, kcache_groups=Kcache)
        e[3].record()
        qd.copy_(Qg[:, :, -1])
        atf.atf_decode(qd, Kcache, V, table=Wuse, O=Od)
        e[4].record()
        if timed:
            torch.cuda.synchronize()
            t_rope.append(e[1].elapsed_time(e[2]))
            t_pre.append(e[2].elapsed_time(e[3]))
            t_dec.append(e[3].elapsed_time(e[4]))
        return W

    for _ in range(args.warmup):
        W = step(False)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    torch.cuda.synchronize()
    wall0 = time.time()
    t0, t1 = ev(), ev()
    t0.record()
    for _ in range(args.steps):
        W = step(True)
    t1.record()
    torch.cuda.synchronize()
    wall1 = time.time()
    total_ms = t0.elapsed_time(t1)
    if world > 1:
        dist.barrier()
        total_ms = max_over_ranks(total_ms, dev)
    atf.binding.check_status()
    pre_ms_all = max_over_ranks(statistics.median(t_pre), dev) if world > 1 else statistics.median(t_pre)
    if rank != 0:
        return
    clocks = sampler.summary(wall0, wall1)

    if args.profile_only:
        sampler.stop()
        print(json.dumps({"profile_only": True, "workload": args.workload, "ms_per_step": total_ms / args.steps,
                          "prefill_ms": statistics.median(t_pre), "decode_us": statistics.median(t_dec) * 1e3}))
        return
    Wl = list(W.arr)
    executed, effective = prefill_flops(wl, Wl)
    issued = prefill_issued_flops(wl, Wl)
    pre_ms = pre_ms_all
    dec_ms = statistics.median(t_dec)
    rope_ms = statistics.median(t_rope)
    step_ms = total_ms / args.steps
    work_ms = rope_ms + pre_ms + dec_ms  # the step's own work, without the copies that restore the un-rotated inputs

    # ---- the same library at k = infinity and in coarse mode, interleaved with the windowed call: each repetition
    #      times the three back to back, so clock drift hits them alike; the ratios are taken per repetition ----
    arms = {"win": dict(table=W), "full": dict(table=None), "coarse": dict(table=W, mode=atf.ATF_MODE_COARSE)}
    ms = {k: [] for k in arms}
    windows = {k: [] for k in arms}
    for k, kw in arms.items():  # warm-up of each arm
        atf.atf_prefill(Qg, Kg, V, O=O, LSE=LSE, **kw)
    torch.cuda.synchronize()
    order = list(arms)
    for rep in range(args.reps):
        for k in order[rep % 3:] + order[:rep % 3]:  # rotate the order: no arm always runs behind the same one
            kw = arms[k]
            a, b_ = ev(), ev()
            w0 = time.time()
            a.record()
            atf.atf_prefill(Qg, Kg, V, O=O, LSE=LSE, **kw)
            b_.record()
            torch.cuda.synchronize()
            windows[k].append((w0, time.time()))
            ms[k].append(a.elapsed_time(b_))
    full_pre_ms, coarse_pre_ms, win_pre_ms = (statistics.median(ms[k]) for k in ("full", "coarse", "win"))
    ratio_win = spread([f / w for f, w in zip(ms["full"], ms["win"])])
    ratio_coarse = spread([f / c for f, c in zip(ms["full"], ms["coarse"])])
    arm_mhz = {k: sampler.mhz_in(windows[k]) for k in arms}
    arm_ms_mhz = {k: (statistics.median(ms[k]) * arm_mhz[k] if arm_mhz[k] else None) for k in arms}

    # ---- the last half of the prompt as appended rows (App. C: the reduction is higher for late rows) ----
    Qh = Qg[:, :, wl.N // 2:].contiguous()
    Oh2 = torch.empty_like(Qh)
    half_pre = []
    for i in range(4):
        a, b_ = ev(), ev()
        a.record()
        atf.atf_prefill(Qh, Kg, V, table=W, O=Oh2, return_lse=False)
        b_.record()
        torch.cuda.synchronize()
        if i:
            half_pre.append(a.elapsed_time(b_))
    half_pre_ms = statistics.median(half_pre)
    del Qh, Oh2
    half_exec, _ = prefill_flops(wl, Wl, n0=wl.N // 2)

    _, theta = atf.atf_window_table(wl.base, wl.d, wl.k, wl.N, wl.scaling)
    dec = time_decode(atf, wl, W, Wl, qd, Kg, V, Kcache, Od, theta)
    dbytes, dbytes_full, dfetch = dec["alg_bytes"], dec["full_bytes"], dec["fetched_bytes"]
    dec_us, dec_full_us, dec_grp_us = dec["rows_us"], dec["rows_full_us"], dec["groups_us"]

    # ---- end to end through the public API with HOST buffers (pinned), copies inside the timed region ----
    hQ, hK, hV = (t.cpu().pin_memory() for t in (Qg, Kg, V))
    Oh = torch.empty(hQ.shape, dtype=torch.bfloat16, pin_memory=True)   # result buffers a caller keeps
    Lh = torch.empty(hQ.shape[:3], dtype=torch.float32, pin_memory=True)
    e2e_t = []
    for i in range(4):
        torch.cuda.synchronize()
        ta = time.perf_counter()
        Oh, Lh = atf.atf_prefill(hQ, hK, hV, table=W, O=Oh, LSE=Lh)
        torch.cuda.synchronize()
        if i:
            e2e_t.append((time.perf_counter() - ta) * 1e3)
    e2e_ms = statistics.median(e2e_t)
    h2d = (hQ.numel() + hK.numel() + hV.numel()) * 2
    d2h = Oh.numel() * 2 + Lh.numel() * 4
    sampler.stop()

    # ---- CPU baseline: the oracle as it stands on a bounded sample of the same workload ----
    cpu = cpu_baseline(wl, budget_s=args.cpu_budget)

    out = {
        "metric": METRIC, "value": aggregate_value(executed, world, pre_ms), "unit": "TFLOP/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{wl.name} attention layer B={wl.B} Hq={wl.Hq} Hkv={wl.Hkv} d={wl.d} N=L={wl.N} k={wl.k} "
                               f"({'llama3-scaled' if wl.scaling else 'raw'} RoPE base {wl.base:g}), exact mode",
                   "step": "window_table + rope(Q,K) + prefill (writes the group-major K cache) + decode on that cache",
                   "l2": "inputs larger than L2; decode alone cycles a KV pool >= 512 MiB, 8 launches per timed region",
                   "replicas": world},
        "prefill_ms": pre_ms, "prefill_executed_tflops": executed / (pre_ms * 1e-3) / 1e12,
        "prefill_effective_tflops": effective / (pre_ms * 1e-3) / 1e12,
        "prefill_issued_tflops": issued / (pre_ms * 1e-3) / 1e12,
        "prefill_interleaved": {"reps": args.reps, "windowed_ms": spread(ms["win"]), "full_ms": spread(ms["full"]),
                                "coarse_ms": spread(ms["coarse"]), "sm_mhz": arm_mhz, "ms_x_mhz": arm_ms_mhz},
        "prefill_full_ms": full_pre_ms, "prefill_speedup_vs_full": ratio_win["median"],
        # the same kernel at k = infinity executes every term: its rate says how close the kernel comes to the
        # tensor peak when the window takes nothing away (the windowed run executes fewer FLOPs in about the same time)
        "prefill_full_executed_tflops": effective / (full_pre_ms * 1e-3) / 1e12,
        "prefill_full_frac_of_peak": effective / (full_pre_ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
        "prefill_speedup_vs_full_spread": ratio_win,
        "prefill_full_tflops": effective / (full_pre_ms * 1e-3) / 1e12,
        "prefill_coarse_ms": coarse_pre_ms, "prefill_coarse_speedup_vs_full": ratio_coarse["median"],
        "prefill_coarse_speedup_vs_full_spread": ratio_coarse,
        "prefill_last_half_ms": half_pre_ms, "prefill_last_half_executed_tflops": half_exec / (half_pre_ms * 1e-3) / 1e12,
        "prefill_ceiling": effective / executed,
        "rope_ms": rope_ms, "work_ms": work_ms,
        # decode on the group-major cache the prefill wrote (the pipeline's path); alone, cycling the pool
        "decode_us": dec_grp_us, "decode_gbs": dbytes / (dec_grp_us * 1e-6) / 1e9,
        "decode_speedup_vs_full": dec_full_us / dec_grp_us, "decode_in_step_us": dec_ms * 1e3,
        # the same step on a position-independent (unrotated) cache: the kernel rotates what it fetches (App. B)
        "decode_rotate_at_read_us": dec["groups_rot_us"],
        # decode on the row-layout cache (atf_decode's default): every K row is read whole, so the window saves no traffic
        "decode_rows_us": dec_us, "decode_rows_gbs": dbytes / (dec_us * 1e-6) / 1e9,
        "decode_full_us": dec_full_us, "decode_full_gbs": dbytes_full / (dec_full_us * 1e-6) / 1e9,
        "decode_rows_speedup_vs_full": dec_full_us / dec_us,
        "frac_of_nominal": {"prefill_executed_of_2250": executed / (pre_ms * 1e-3) / 1e12 / 2250.0,
                            "decode_of_8000": dbytes / (dec_grp_us * 1e-6) / 1e9 / 8000.0},
        "roofline": {"bound": "tensor", "achieved": executed / (pre_ms * 1e-3) / 1e12,
                     "peak": pk["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": executed / (pre_ms * 1e-3) / 1e12 / pk["bf16_tflops_sustained"],
                     # DRAM bytes of one launch: ncu capture at N = 32768 (511 MB) scaled by N (traffic is the
                     # repacked Q/K, V and O once each, linear in N)
                     "traffic": 511.7e6 * wl.N / 32768 if wl.name == "llama-3.2-3b" else None,
                     "kernel": "atf_prefill_pipe_kernel (+ schedule and 2 repack launches, <1% of the time)",
                     "peak_source": f"{pk['source']} sustained bf16 GEMM"},
        "roofline_decode": {"bound": "hbm", "achieved": dbytes / (dec_grp_us * 1e-6) / 1e9, "peak": pk["hbm_gbs"],
                            "unit": "GB/s", "frac": dbytes / (dec_grp_us * 1e-6) / 1e9 / pk["hbm_gbs"],
                            # bytes the launch asks for: live groups of 8 pairs per 64-key tile + V
                            "traffic": float(dfetch),
                            "achieved_bytes_read": dfetch / (dec_grp_us * 1e-6) / 1e9,
                            "frac_bytes_read": dfetch / (dec_grp_us * 1e-6) / 1e9 / pk["hbm_gbs"],
                            "kernel": "atf_decode_tiles_kernel (group-major K cache)",
                            "peak_source": f"{pk['source']} copy bandwidth"},
        "e2e": {"value": executed / (e2e_ms * 1e-3) / 1e12, "unit": "TFLOP/s", "ms": e2e_ms,
                "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                "what": "atf_prefill on pinned host tensors = the C call atf_prefill_host: H2D of Q,K,V, kernels and D2H of O,LSE, overlapped chunk by chunk (16K rows) on three streams"},
        "gpu_launches": 7 * args.steps,  # per step: 2 rope + schedule + 2 repack + prefill + decode
        "clocks": clocks,
        "cpu_baseline": cpu,
    }
    print(json.dumps(out))


def time_decode(atf, wl, W, Wl, qd, Kg, V, Kcache, Od, theta):
    """Decode alone, cycling a KV pool of >= 512 MiB so that no read hits L2 from an earlier one.  Each timed
    region holds DEC_BATCH launches back to back (one per pool entry in turn), so the device queue stays full and
    the host's call overhead (~15 us per call through the binding) is not billed to the kernel.
    The "rot" arm is the rotate-at-read decode (App. B) on the same group-major bytes taken as unrotated keys: its
    cost does not depend on the values."""
    kv_bytes = 2 * Kg.numel() * 2
    npool = max(2, math.ceil((512 << 20) / kv_bytes) + 1)
    pool = [(Kg, V)] + [(Kg.clone(), V.clone()) for _ in range(npool - 1)]
    gpool = [Kcache] + [Kcache.clone() for _ in range(npool - 1)]  # the caches the prefill wrote, group-major
    DEC_BATCH = 8
    tabs = atf.atf_rope_tables(theta, wl.d, Kcache.shape[2] * Kcache.shape[4], device=qd.device)
    dec_t = {"win": [], "full": [], "grp": [], "rot": []}
    for kind in ("win", "full", "grp", "rot"):
        it = 0
        for rep in range(2 + 10):
            a, b_ = ev(), ev()
            a.record()
            for _ in range(DEC_BATCH):
                Kc, Vc = pool[it % npool]
                if kind in ("grp", "rot"):
                    Kc = gpool[it % npool]
                it += 1
                atf.atf_decode(qd, Kc, Vc, table=None if kind == "full" else W, O=Od,
                               rope_tables=tabs if kind == "rot" else None)
            b_.record()
            torch.cuda.synchronize()
            if rep >= 2:
                dec_t[kind].append(a.elapsed_time(b_) * 1e3 / DEC_BATCH)
    atf.binding.check_status()
    return {"rows_us": statistics.median(dec_t["win"]), "rows_full_us": statistics.median(dec_t["full"]),
            "groups_us": statistics.median(dec_t["grp"]), "groups_rot_us": statistics.median(dec_t["rot"]), "alg_bytes": decode_bytes(wl, Wl, True),
            "full_bytes": decode_bytes(wl, Wl, False), "fetched_bytes": decode_fetched_bytes(wl, Wl)}


def run_decode_only(args, atf, wl, pk, dev):
    """Decode configurations that have no prefill of their own (B = 8): post-RoPE caches drawn directly, the
    group-major cache written by the pack call; prints a short line (sweep files under profiles/)."""
    q, Kc, Vc = gen.decode_inputs(wl, device=dev)
    W, theta = atf.atf_window_table(wl.base, wl.d, wl.k, wl.N, wl.scaling)
    Wl = W.tolist()
    Wt = atf.WindowTable(W)
    atf.ensure_workspace(atf.atf_workspace_bytes(1, wl.B, wl.Hq, wl.Hkv, wl.N, wl.d), dev)
    Kcache = atf.atf_kcache_pack(Kc)
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    w0 = time.time()
    d = time_decode(atf, wl, Wt, Wl, q, Kc, Vc, Kcache, torch.empty_like(q), theta)
    clocks = sampler.summary(w0, time.time())
    sampler.stop()
    print(json.dumps({"decode_only": True, "workload": args.workload, "B": wl.B, "L": wl.N,
                      "groups_us": d["groups_us"], "groups_gbs": d["alg_bytes"] / d["groups_us"] / 1e3,
                      "groups_frac_of_hbm": d["alg_bytes"] / d["groups_us"] / 1e3 / pk["hbm_gbs"],
                      "rows_us": d["rows_us"], "rows_full_us": d["rows_full_us"], "groups_rot_us": d["groups_rot_us"],
                      "groups_speedup_vs_full": d["rows_full_us"] / d["groups_us"],
                      "alg_MB": d["alg_bytes"] / 1e6, "fetched_MB": d["fetched_bytes"] / 1e6, "full_MB": d["full_bytes"] / 1e6,
                      "clocks": clocks}))


def run_split_precision(args, atf, wl, dev):
    """Cost of the split-precision prefill (fp32 Q/K, three tensor-core products per score step) beside the bf16
    path on the same rotated values; prints a short line (sweep file under profiles/)."""
    W, theta = atf.atf_window_table(wl.base, wl.d, wl.k, wl.N, wl.scaling)
    Wt = atf.WindowTable(W)
    Q, K, V = gen.prefill_inputs_f32(wl, device=dev)
    atf.atf_rope_f32(Q, theta)
    atf.atf_rope_f32(K, theta)
    Qb, Kb = Q.to(torch.bfloat16), K.to(torch.bfloat16)
    O = torch.empty(Q.shape, dtype=torch.bfloat16, device=dev)
    LSE = torch.empty(Q.shape[:3], dtype=torch.float32, device=dev)
    atf.ensure_workspace(atf.atf_workspace_bytes(atf.ATF_OP_PREFILL_SPLIT, wl.B, wl.Hq, wl.Hkv, wl.N, wl.d), dev)
    arms = {"split_exact_ms": lambda: atf.atf_prefill_split(Q, K, V, table=Wt, O=O, LSE=LSE),
            "split_coarse_ms": lambda: atf.atf_prefill_split(Q, K, V, table=Wt, O=O, LSE=LSE, mode=atf.ATF_MODE_COARSE),
            "split_full_ms": lambda: atf.atf_prefill_split(Q, K, V, table=None, O=O, LSE=LSE),
            "bf16_exact_ms": lambda: atf.atf_prefill(Qb, Kb, V, table=Wt, O=O, LSE=LSE),
            "bf16_coarse_ms": lambda: atf.atf_prefill(Qb, Kb, V, table=Wt, O=O, LSE=LSE, mode=atf.ATF_MODE_COARSE),
            "bf16_full_ms": lambda: atf.atf_prefill(Qb, Kb, V, table=None, O=O, LSE=LSE)}
    sampler = ClockSampler(dev.index or 0)
    sampler.start()
    w0 = time.time()
    ts = {k: [] for k in arms}
    for rep in range(2 + 5):        # interleaved, inputs larger than L2 at the sizes this is quoted on
        for k, fn in arms.items():
            a, b_ = ev(), ev()
            a.record()
            fn()
            b_.record()
            torch.cuda.synchronize()
            if rep >= 2:
                ts[k].append(a.elapsed_time(b_))
    clocks = sampler.summary(w0, time.time())
    sampler.stop()
    atf.binding.check_status()
    out = {"split_precision": True, "workload": args.workload, "N": wl.N}
    out.update({k: statistics.median(v) for k, v in ts.items()})
    out["split_over_bf16_exact"] = out["split_exact_ms"] / out["bf16_exact_ms"]
    out["split_over_bf16_coarse"] = out["split_coarse_ms"] / out["bf16_coarse_ms"]
    out["split_window_speedup_exact"] = out["split_full_ms"] / out["split_exact_ms"]
    out["split_window_speedup_coarse"] = out["split_full_ms"] / out["split_coarse_ms"]
    out["clocks"] = clocks
    print(json.dumps(out))


def run_probe_lines(args):
    """What DRAM moves when parts of 256-byte rows are left out (the library's read diagnostic): one line per mask."""
    import paper_2608_02947_b200 as atf
    dev = torch.device("cuda", int(os.environ.get("LOCAL_RANK", "0")))
    torch.cuda.set_device(dev)
    atf.ensure_workspace(1 << 20, dev)
    buf = torch.ones(1 << 30, dtype=torch.uint8, device=dev)
    for mask in (0xFFFF, 0xF0F0, 0xFCFC, 0xFF00, 0x00FF, 0xF000):
        best = 1e9
        for rep in range(6):
            a, b_ = ev(), ev()
            a.record()
            atf.binding.probe_masked_read(buf, mask)
            b_.record()
            torch.cuda.synchronize()
            if rep:
                best = min(best, a.elapsed_time(b_))
        live = bin(mask).count("1")
        print(json.dumps({"probe_lines": True, "mask": f"{mask:04x}", "live_chunks_of_16": live, "ms": best,
                          "requested_GB": buf.numel() * live / 16 / 1e9,
                          "requested_GBps": buf.numel() * live / 16 / best / 1e6,
                          "whole_rows_GBps": buf.numel() / best / 1e6}))


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return {p.get("internal_api", p.get("user_api", "?")): p.get("num_threads") for p in threadpool_info()}
    except Exception:
        return None


def cpu_baseline(wl, budget_s=15.0):
    """Times oracle/ (fp64 NumPy, as it stands) on sampled query rows of the same workload."""
    import numpy as np

    from oracle import atf_oracle as orc
    W, theta = orc.window_table(wl.base, wl.d, wl.k, wl.N, wl.scaling)
    rng = np.random.default_rng(wl.seed)
    # one head's worth of rotated-looking data (the cost does not depend on values)
    K = orc.round_to_bf16(rng.standard_normal((wl.N, wl.d)))
    V = orc.round_to_bf16(rng.standard_normal((wl.N, wl.d)))
    Q = orc.round_to_bf16(rng.standard_normal((wl.N, wl.d)))
    rows, flops = 0, 0
    t0, c0 = time.perf_counter(), time.process_time()
    while time.perf_counter() - t0 < budget_s:
        n = int(rng.integers(0, wl.N))
        orc.attention_rows(Q, K, V, W, [n])
        rows += 1
        flops += 4 * orc.kept_terms_row(W, n) + 2 * wl.d * (n + 1)
    dt, cpu_s = time.perf_counter() - t0, time.process_time() - c0
    used = max(1, round(cpu_s / dt))  # threads the oracle actually kept busy (CPU time / wall time)
    return {"value": flops / dt / 1e12, "unit": "TFLOP/s", "cores": used, "kind": "oracle",
            "sample": f"{rows} random query rows of one head of the {wl.N}-token workload in {dt:.1f} s "
                      f"(fp64 NumPy; CPU time / wall time = {cpu_s / dt:.2f}); executed FLOPs of those rows / time",
            "host_cores_available": os.cpu_count(), "blas_threads": blas_threads()}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    wl = workload_by_name(args.workload)
    vals = []
    per = max(2.0, min(20.0, 120.0 / max(1, args.steps + args.warmup)))
    for i in range(args.warmup + args.steps):
        c = cpu_baseline(wl, budget_s=per)
        if i >= args.warmup:
            vals.append(c)
    v = statistics.median([c["value"] for c in vals])
    out = {"impl": "reference", "metric": METRIC, "value": v, "unit": "TFLOP/s", "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": f"{wl.name} attention layer N={wl.N} (bounded sample of query rows per step)"},
           "cpu_baseline": {"value": v, "unit": "TFLOP/s", "cores": vals[-1]["cores"], "kind": "oracle",
                            "sample": vals[-1]["sample"], "blas_threads": vals[-1]["blas_threads"]},
           "e2e": {"value": v, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def run_replica_selftest(args):
    """Host logic of the replica launch without a GPU: every rank reports a made-up time, rank 0 prints the
    aggregate of the slowest one (gloo).  Used by the CPU tests of `--gpus N`."""
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    ms = max_over_ranks(10.0 + 5.0 * rank, torch.device("cpu"))
    if world > 1:
        dist.barrier()
    if rank == 0:
        print(json.dumps({"replica_selftest": True, "n_gpus": world, "ms": ms,
                          "value": aggregate_value(3.0e12, world, ms)}))


def spawn_replicas(args):
    """`python bench.py --gpus N` outside a launcher: start the N ranks (one process per GPU) the way the launcher
    would, on this node, and pass their output through."""
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    raise SystemExit(subprocess.run(cmd, env=env).returncode)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--reps", type=int, default=12, help="interleaved repetitions of windowed / k = infinity / coarse")
    ap.add_argument("--impl", default="ours")
    ap.add_argument("--workload", default="llama3b-128k")
    ap.add_argument("--cpu-budget", type=float, default=15.0)
    ap.add_argument("--full-attention", action="store_true",
                    help="run the step with table = NULL (the library's own k = infinity mode)")
    ap.add_argument("--decode-only", action="store_true",
                    help="time only decode on the workload's cache shape (for the B = 8 configurations)")
    ap.add_argument("--split-precision", action="store_true",
                    help="time the split-precision prefill beside the bf16 path on the workload's shape")
    ap.add_argument("--profile-only", action="store_true",
                    help="run only the warm-up and timed steps (for profiler captures); prints a short line")
    ap.add_argument("--probe-lines", action="store_true",
                    help="time the library's masked row-read diagnostic (DRAM line granularity) and exit")
    ap.add_argument("--replica-selftest", action="store_true", help=argparse.SUPPRESS)
    args = ap.parse_args()
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        spawn_replicas(args)
    if args.probe_lines:
        run_probe_lines(args)
    elif args.replica_selftest:
        run_replica_selftest(args)
    elif args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()

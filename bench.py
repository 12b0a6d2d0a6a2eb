#!/usr/bin/env python
"""Benchmark of the MLA-Online layer (RedKnot-MLA, Algorithm 2) on B200.

One step = one pass of the whole hot path over one synthetic request:
rk_mla_online_attn (relocation fused, segments merged in-kernel) -> rk_group_sliced_proj ->
rk_combine_offline (restore-and-replace + shared W_b).  Metric: prefill tokens/s per layer.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl reference]

With N > 1 every rank runs its own independent request of the same shape (the path has no exchange
step: weak scaling, no collective in the data path); the value is the total over ranks divided by the
slowest rank's device time.  Started under torch.distributed.run the ranks come from the environment;
started plainly with --gpus N > 1 the script starts the N ranks itself (one process per GPU,
rendezvous on 127.0.0.1) and rank 0 prints the one JSON line.
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
sys.path.insert(0, ROOT)

from paper_2609_07008_b200 import synth  # noqa: E402
from paper_2609_07008_b200 import dist as rkdist  # noqa: E402

FLOP_PER_PAIR = 2 * 576 + 2 * 512     # QK^T over 576 + PV over 512 per visible (row, key, head)
# dram__bytes_read.sum + dram__bytes_write.sum of the attention kernel's two launches per step, from the
# one-pass ncu captures summarised under profiles/ (bytes per step; None where no capture exists).  bench.py
# cannot run ncu itself: the figure is the capture's, taken on the kernel named in `captured_on`.
PROFILED_DRAM_TRAFFIC = {
    "flash256k": dict(bytes=37.41e9 + 9.24e9, algorithmic=4.91e9 + 1.20e9,
                      source="profiles/attn_kernel_flash256k_dram_traffic.md",
                      captured_on="commit 4117a6a: rk_mla_attn_kernel<kPhase=0, kStarve=0> (unchanged since for this instantiation)"),
    "flash1": dict(bytes=(352.5e6 + 224.8e6) + (169.3e6 + 74.4e6), algorithmic=(350.3e6 + 277.9e6) + (168.4e6 + 115.5e6),
                   source="profiles/attn_kernel_flash1_ncu_full.md",
                   captured_on="commit 4117a6a: rk_mla_attn_kernel<kPhase=0, kStarve=0> (unchanged since for this instantiation)"),
}
# Tensor-pipe use counted in SM cycles, from the one-pass ncu capture of the SM clock during the two attention launches
# (profiles/attn_kernel_flash256k_sm_clock.md): rate / (148 SMs x 8192 flop per clock x measured clock).  A capture's
# figure, like the traffic above; the NVML clock samples the bench takes itself overstate the clock the kernels get.
PROFILED_PIPE_USE = {
    "flash256k": dict(global_pass=0.935, local_pass=0.949, sm_ghz_global=1.317, sm_ghz_local=1.381,
                      source="profiles/attn_kernel_flash256k_sm_clock.md"),
}
L2_BYTES = 126 * 1024 * 1024


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_burst=d["bf16_tflops"], bf16_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_burst=1590.0, bf16_sustained=1400.0, source="fallback")


class ClockSampler(threading.Thread):
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.stop_flag = index, [], False

    def run(self):
        while not self.stop_flag:
            try:
                out = subprocess.run(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                      "-i", str(self.index)], capture_output=True, text=True, timeout=5).stdout
                f = [x.strip() for x in out.strip().split(",")]
                if len(f) >= 6:
                    self.samples.append(f)
            except Exception:
                pass
            time.sleep(0.2)

    def summary(self):
        if not self.samples:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["unavailable"])
        mhz = sorted(int(s[0]) for s in self.samples if s[0].isdigit())
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(s[2 + i].lower().startswith("active") for s in self.samples)]
        return dict(sm_mhz=mhz[len(mhz) // 2] if mhz else None, sm_max_mhz=int(self.samples[0][1]), reasons=reasons,
                    samples=len(self.samples))


class NvmlClock(threading.Thread):
    """SM clock of one GPU read through NVML every few milliseconds (nvidia-smi is too slow for a region of a
    few hundred milliseconds).  Read-only: nothing is set."""

    def __init__(self, index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.index, self.period, self.samples, self.stop_flag, self.ok = index, period_s, [], False, False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            self.max_mhz = None

    def run(self):
        while self.ok and not self.stop_flag:
            try:
                self.samples.append(int(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM)))
            except Exception:
                pass
            time.sleep(self.period)

    def median(self):
        v = sorted(self.samples)
        return v[len(v) // 2] if v else None


AUX_SCALE = 1.0      # --aux-scale: shortens the steady-state loops (profiler runs)


def timed_region(fn, stream, gpu_index, min_ms=300.0, lead_ms=30.0):
    """Times one call `fn` in its steady state: the same call is first repeated for at least lead_ms, then
    timed back to back (CUDA events on the launching stream) over at least 20 repeats and min_ms, with the
    SM clock sampled through NVML during the timed repeats.  Returns (ms per call, median SM MHz, max SM MHz)."""
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    fn()
    b.record(stream)
    torch.cuda.synchronize()
    one = max(a.elapsed_time(b), 1e-3)
    for _ in range(max(3, int(lead_ms * AUX_SCALE / one))):
        fn()
    reps = max(20 if AUX_SCALE >= 1.0 else 3, int(min_ms * AUX_SCALE / one))
    clk = NvmlClock(gpu_index)
    torch.cuda.synchronize()
    clk.start()
    a.record(stream)
    for _ in range(reps):
        fn()
    b.record(stream)
    torch.cuda.synchronize()
    clk.stop_flag = True
    clk.join(timeout=1)
    return a.elapsed_time(b) / reps, clk.median(), clk.max_mhz


def hbm_entry(ms, nbytes, mhz, max_mhz, **kw):
    """One standalone HBM-bound kernel: GB/s as measured, the SM clock it ran at, and GB/s scaled to the maximum
    clock (what an issue- or latency-bound kernel would read at full clock; a DRAM-bound one does not scale)."""
    gbs = nbytes / ms / 1e6
    d = dict(ms=ms, bytes=nbytes, gbs=gbs, sm_mhz=mhz, sm_max_mhz=max_mhz, **kw)
    if mhz and max_mhz:
        d["gbs_at_max_clock"] = gbs * max_mhz / mhz
    return d


def algorithmic_flops(profile, req, value_phase=False):
    """Work the method itself must do: Global heads x all rows + Local heads x protected rows.  In the
    output-phase variant the value is the whole 576-wide row: 2*576 + 2*576 flop per visible pair and a
    576-wide W_uv."""
    G, L, ro, dm = profile.n_groups, profile.n_local, profile.o_rank, profile.d_model
    ow = 576 if value_phase else 512
    attn = (2 * 576 + 2 * ow) * (G * req.pairs_global + L * req.pairs_local)
    proj = 2 * req.T * G * (ow * 128 + 128 * ro) + 2 * req.A * (L * ow * 128 + G * 7 * 128 * ro)
    wb = 2 * req.T * G * ro * dm
    return attn, proj, wb


# ------------------------------------------------------------------------------------------------
# CPU checker timing (cpu_baseline leg and --impl reference)
# ------------------------------------------------------------------------------------------------

def oracle_sample_run(w, rows, value_phase=False):
    """Runs the float64 checker on the packed rows `rows`; returns (seconds, visible pairs)."""
    import oracle
    from oracle.harness import f64
    p, lay = w.profile, w.layout
    rows = np.asarray(rows, dtype=np.int64)
    inv = oracle.inverse_row_map(w.prot_rows, lay.n_rows)
    ridx = torch.as_tensor(rows, device=w.q_g.device)
    q_g_rows = f64(w.q_g[ridx])
    ql = {int(r): f64(w.q_l[int(inv[r])]) for r in rows if inv[r] >= 0}
    zo = {int(r): f64(w.z_off[int(r)]) for r in rows if inv[r] < 0}
    kv, wuv, wa, wb = f64(w.kv), f64(w.w_uv), f64(w.w_a), f64(w.w_b)
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    srt = np.sort(pos)
    vis = np.searchsorted(srt, pos[rows], side="right")
    pairs = int(sum(v * (p.n_heads if inv[r] >= 0 else p.n_groups) for v, r in zip(vis, rows)))
    t0 = time.perf_counter()
    fn = oracle.phase.mla_online_rows_phase if value_phase else oracle.mla_online_rows
    out = fn(rows, q_g_rows, ql, kv, lay.seg_off, lay.seg_delta, w.prot_rows, p.global_heads,
             p.local_heads, wuv, wa, wb, zo, p.sm_scale, p.rope_base, p.d_latent)
    dt = time.perf_counter() - t0
    return dt, pairs, out


def pick_oracle_rows(w, pair_budget):
    """Seeded sample of rows (half protected) whose visible-pair count stays within the budget."""
    p, lay = w.profile, w.layout
    cand = synth.sample_rows(lay, w.prot_rows, 64, w.seed)
    import oracle
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    srt = np.sort(pos)
    inv = oracle.inverse_row_map(w.prot_rows, lay.n_rows)
    rng = np.random.default_rng(w.seed + 5)
    cand = rng.permutation(cand)
    rows, used = [], 0
    for r in cand:
        c = int(np.searchsorted(srt, pos[r], side="right")) * (p.n_heads if inv[r] >= 0 else p.n_groups)
        if used + c > pair_budget and rows:
            continue
        rows.append(int(r))
        used += c
        if used >= pair_budget:
            break
    return np.sort(np.asarray(rows, dtype=np.int64))


def total_pairs(profile, req):
    return profile.n_groups * req.pairs_global + profile.n_local * req.pairs_local


def run_reference(args, rank, world):
    """--impl reference: the float64 CPU checker, as it stands, on the host cores; every step is
    a bounded row sample of the same workload and tokens/s is extrapolated by visible pairs."""
    if rank != 0:
        return
    name = args.config
    prof, lay, prot = synth.make_geometry(name)
    w = synth.make_tensors(name, prof, lay, prot, synth.CONFIGS[name]["seed"] * 1000, device="cpu",
                           value_phase=args.value_phase)
    import oracle
    pos = oracle.request_positions(lay.seg_off, lay.seg_delta)
    srt = np.sort(pos)
    pg = int(np.searchsorted(srt, pos, side="right").sum())
    pl = int(np.searchsorted(srt, pos[prot], side="right").sum())
    all_pairs = prof.n_groups * pg + prof.n_local * pl
    # every step is one bounded sample; a third of the cpu_baseline budget keeps W + K steps within minutes
    rows = pick_oracle_rows(w, max(1, args.oracle_pairs // 3))
    times, pairs = [], 0
    for i in range(args.warmup + args.steps):
        dt, pairs, _ = oracle_sample_run(w, rows, args.value_phase)
        if i >= args.warmup:
            times.append(dt)
    sec = float(np.mean(times))
    tok_s = lay.n_rows / (sec * all_pairs / pairs)
    cores = os.cpu_count()
    line = dict(metric="mla_online_prefill_tokens_per_s_per_layer", value=tok_s, unit="tokens/s", n_gpus=world,
                steps=args.steps, warmup=args.warmup, ms_per_step=sec * 1e3 * all_pairs / pairs,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                impl="reference", config=dict(workload=name, T=lay.n_rows, n_prot=len(prot), value_phase=args.value_phase),
                cpu_baseline=dict(value=tok_s, unit="tokens/s", cores=cores, kind="oracle",
                                  sample=f"{len(rows)} seeded rows, {pairs} of {all_pairs} visible (row,key,head) "
                                         f"pairs per step, extrapolated by pair count"),
                e2e=dict(value=tok_s, unit="tokens/s", h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------

def time_stream_kernels(ctx, req, w, prof, lay, dev, budget_bytes=6 << 30):
    """rk_relocate_q over (rows x Global heads x frames) and rk_segmented_merge over
    (query-suffix rows x all heads x parts), each sized to a few GB (far beyond L2), timed in their steady
    state (see timed_region); algorithmic bytes = every tensor read or written once."""
    res = {}
    stream = torch.cuda.current_stream()
    gpu = dev.index or 0

    G, S, T = prof.n_groups, lay.n_segs, lay.n_rows
    frame_bytes = T * G * 64 * 2
    frames = int(max(1, min(S, budget_bytes // frame_bytes)))
    out = torch.empty((frames, T, G, 64), dtype=torch.bfloat16, device=dev)
    view = w.q_g[:, :, 512:]
    ms, mhz, mx = timed_region(lambda: ctx.rk_relocate_q(req, view, 0, frames, out), stream, gpu)
    nbytes = frame_bytes * (1 + frames)
    res["rk_relocate_q"] = hbm_entry(ms, nbytes, mhz, mx, frames=frames, rows=T, heads=G)
    del out
    H = prof.n_heads
    n_q = int(lay.seg_off[-1] - lay.seg_off[-2])
    part_bytes = n_q * H * (512 * 2 + 4)
    parts = int(max(2, min(S, budget_bytes // part_bytes)))
    O_part = torch.randn((parts, n_q, H, 512), device=dev, dtype=torch.float32).to(torch.bfloat16)
    lse_part = torch.randn((parts, n_q, H), device=dev, dtype=torch.float32)
    O = torch.empty((n_q, H, 512), dtype=torch.bfloat16, device=dev)
    lse = torch.empty((n_q, H), dtype=torch.float32, device=dev)
    ms, mhz, mx = timed_region(lambda: ctx.rk_segmented_merge(O_part, lse_part, O, lse), stream, gpu)
    nbytes = part_bytes * parts + n_q * H * (512 * 2 + 4)
    res["rk_segmented_merge"] = hbm_entry(ms, nbytes, mhz, mx, parts=parts, rows=n_q, heads=H)
    ctx.rk_poll_status()
    return res


def time_selection_rules(ctx, lay, dev):
    """rk_protected_rows on the bench request with the paper's constants at the 25 % budget (flag pass,
    8 select passes, 3 compaction passes; the time is launch latency, the bytes are a few per row) and
    rk_moe_fanout on 16 M tokens (26 B per token, a plain streaming pass)."""
    from paper_2609_07008_b200 import synth as _synth
    stream = torch.cuda.current_stream()
    gpu = dev.index or 0

    res = {}
    dirty, scores = _synth.draw_policy_inputs(lay, seed=99, n_dirty=500)
    d, s = torch.from_numpy(dirty).to(dev), torch.from_numpy(scores).to(dev)
    T, S = lay.n_rows, lay.n_segs
    out = ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, d, s, budget_bp=2500)
    ws = torch.empty(16 << 20, dtype=torch.uint8, device=dev)
    ms, mhz, mx = timed_region(lambda: ctx.rk_protected_rows(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, d, s,
                                                             budget_bp=2500, out=out, workspace=ws), stream, gpu, min_ms=100.0)
    n_sel = int(out[1].item())
    # per row: flag pass 1 B written; 8 select passes 1 B flag + 4 B score; count 5 B; scatter 5 B + output
    nbytes = T * (1 + 8 * 5 + 5 + 5) + 4 * n_sel + 4 * len(dirty)
    res["rk_protected_rows"] = dict(ms=ms, rows=T, selected=n_sel, budget_bp=2500, launches=13, bytes=nbytes,
                                    gbs=nbytes / ms / 1e6, sm_mhz=mhz,
                                    bound="launch latency (13 short kernels + 4 small copies)")
    n = 64 << 20                           # 1.6 GB of router weights: far beyond L2
    p = torch.rand((n, 6), device=dev, dtype=torch.float32) + 0.01
    k, keep = ctx.rk_moe_fanout(p, 0.85)
    ms, mhz, mx = timed_region(lambda: ctx.rk_moe_fanout(p, 0.85, False, k, keep), stream, gpu)
    nbytes = n * 26
    res["rk_moe_fanout"] = hbm_entry(ms, nbytes, mhz, mx, tokens=n)
    ctx.rk_poll_status()
    return res


def time_offline_build(ctx, req, w, prof, lay, dev, rows_per_call=65536):
    """Offline MLA-Off artifact build (Algorithm 1) over every document row, in row ranges; not part of
    the online step.  Flops: 2176 per visible (row, key, Local head) pair inside each document alone,
    plus the Local half of the sliced projection."""
    n, L, G, ro = lay.n_doc_rows, prof.n_local, prof.n_groups, prof.o_rank
    rows_per_call = min(rows_per_call, n)
    q = (torch.randn((rows_per_call, L, 576), device=dev, dtype=torch.float32)).to(torch.bfloat16)
    z = torch.empty((rows_per_call, G * ro), dtype=torch.bfloat16, device=dev)
    import ctypes as C
    from paper_2609_07008_b200 import binding as rk
    ws_n = C.c_size_t()
    rk.lib.rk_mla_off_workspace_bytes(req.handle, rows_per_call, C.byref(ws_n))
    ws = torch.empty(ws_n.value, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()
    pairs = 0
    for i in range(lay.n_segs):
        if lay.seg_has_artifact[i]:
            m = int(lay.seg_off[i + 1] - lay.seg_off[i])
            pairs += m * (m + 1) // 2
    flops = 2176 * L * pairs + 2 * n * (L * 512 * 128 + G * 7 * 128 * ro)

    def run():
        for lo in range(0, n, rows_per_call):
            hi = min(n, lo + rows_per_call)
            ctx.rk_mla_off_build(req, w.kv, lo, hi, q[: hi - lo], w.w_uv, w.w_a, z[: hi - lo], ws)

    ms, mhz, mx = timed_region(run, stream, dev.index or 0, min_ms=300.0, lead_ms=50.0)   # steady state, like the other kernels
    ctx.rk_poll_status()
    return dict(ms=ms, rows=n, tokens_per_s=n / ms * 1e3, tflops=flops / ms / 1e9, rows_per_call=rows_per_call,
                flops=flops, sm_mhz=mhz)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="flash256k", choices=list(synth.CONFIGS))
    ap.add_argument("--impl", default="rk", choices=["rk", "reference"])
    ap.add_argument("--regime", default="mandated", choices=["mandated", "sharp"])
    ap.add_argument("--oracle-pairs", type=int, default=150_000_000,
                    help="visible-pair budget of the CPU checker sample (about 10-30 s of host work)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--protect-bp", type=int, default=None,
                    help="override the share of protected document rows (basis points), e.g. the paper's controller "
                         "budgets 1000 / 2000 / 2500; default: the configuration's own share")
    ap.add_argument("--value-phase", action="store_true",
                    help="the output-phase variant: the whole stored row is the value (RestorePhase per segment and "
                         "the inverse output RoPE inside the attention kernel), W_uv 576 wide")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-aux", action="store_true", help="skip the standalone relocation / merge timings")
    ap.add_argument("--aux-scale", type=float, default=1.0,
                    help="scales the length of the steady-state timing loops of the standalone kernels and of the "
                         "projection breakdown (1 = at least 20 repeats over 150-300 ms; a profiler run uses 0.01)")
    ap.add_argument("--with-offline", action="store_true", help="also time the offline artifact build")
    ap.add_argument("--layers", type=int, default=0,
                    help="independent layer invocations per step (own values and protected rows each; "
                         "default 37 for flash32k, the 3F-37R-3F stack, else 1)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "rk" else args.warmup
    global AUX_SCALE
    AUX_SCALE = args.aux_scale

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started plainly: bring up one rank per GPU ourselves (the same launch torch.distributed.run does)
        sys.exit(rkdist.spawn_ranks(args.gpus, [os.path.abspath(__file__)] + sys.argv[1:]))
    rank, world, local_rank = rkdist.env_ranks()
    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    rkdist.init("nccl", dev)
    from paper_2609_07008_b200 import build as rkbuild
    if local_rank == 0:
        rkbuild.ensure_built()                        # a fresh checkout: compile once with nvcc (no other path exists)
    rkdist.barrier()
    from paper_2609_07008_b200 import binding as rk   # raises if librk.so is missing: no fallback

    name = args.config
    n_layers = args.layers or (synth.N_LAYERS_FLASH32K if name == "flash32k" else 1)
    ctx = None
    layers = []          # (workload, request) per layer: same layout, own values, own protected rows
    for l in range(n_layers):
        prof, lay, prot = synth.make_geometry(name, layer=l, pct_bp=args.protect_bp)
        # every rank gets its own request values (independent requests, same shape)
        wl = synth.make_tensors(name, prof, lay, prot, rkdist.rank_seed(synth.CONFIGS[name]["seed"], rank) + 7 * l,
                                device=dev, regime=args.regime, value_phase=args.value_phase)
        if ctx is None:
            ctx = rk.Context.from_profile(prof, value_phase=args.value_phase)
        layers.append((wl, ctx.rk_request_create(lay.seg_off, lay.seg_delta, lay.seg_has_artifact, prot)))
    w, req = layers[0]
    prof, lay = w.profile, w.layout
    big = max(layers, key=lambda t: t[1].A)[1]
    bufs = ctx.alloc_layer_buffers(big, dev)          # staging/outputs shared by the layers (they run in sequence)
    fl_attn = fl_proj = fl_wb = 0
    for _, r in layers:
        a, b, c = algorithmic_flops(prof, r, args.value_phase)
        fl_attn, fl_proj, fl_wb = fl_attn + a, fl_proj + b, fl_wb + c
    in_bytes = sum(t.numel() * t.element_size() for wl, _ in layers for t in (wl.kv, wl.q_g, wl.q_l, wl.z_off))
    need_flush = in_bytes < 4 * L2_BYTES
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev) if need_flush else None
    stream = torch.cuda.current_stream()

    def run_layer(wl, r, ev=None):
        if ev: ev[0].record(stream)
        ctx.rk_mla_online_attn(r, wl.kv, wl.q_g, None, bufs["O_g"], bufs["lse_g"], None, None)
        if ev: ev[1].record(stream)
        ctx.rk_mla_online_attn(r, wl.kv, None, wl.q_l, None, None, bufs["O_l"], bufs["lse_l"])
        if ev: ev[2].record(stream)
        ctx.rk_group_sliced_proj(r, bufs["O_g"], bufs["O_l"], wl.w_uv, wl.w_a, bufs["z_on_g"], bufs["z_on_l"],
                                 bufs["workspace"])
        if ev: ev[4].record(stream)
        ctx.rk_combine_offline(r, bufs["z_on_g"], bufs["z_on_l"], wl.z_off, wl.w_b, bufs["z"], bufs["y"])
        if ev: ev[3].record(stream)

    def step(ev=None):
        for i, (wl, r) in enumerate(layers):
            run_layer(wl, r, ev[i] if ev else None)

    # per layer: attention x2; sliced projection: Global half fused (1 launch) when r_o is a multiple of 256, else 2,
    # Local half 2; combine; W_b
    launches_per_step = (2 + (1 if prof.o_rank % 256 == 0 else 2) + 2 + 1 + 1) * n_layers

    for _ in range(args.warmup):
        step()
        if need_flush: flush_buf.fill_(1)
    torch.cuda.synchronize()
    ctx.rk_poll_status()

    sampler = ClockSampler(local_rank)
    sampler.start()
    evs = [[[torch.cuda.Event(enable_timing=True) for _ in range(5)] for _ in range(n_layers)]
           for _ in range(args.steps)]
    rkdist.barrier()
    torch.cuda.synchronize()
    for i in range(args.steps):
        step(evs[i])
        if need_flush: flush_buf.fill_(1)
    torch.cuda.synchronize()
    rkdist.barrier()
    sampler.stop_flag = True
    ctx.rk_poll_status()
    step_ms = [evs[i][0][0].elapsed_time(evs[i][-1][3]) for i in range(args.steps)]
    attn_ms = [sum(e[0].elapsed_time(e[2]) for e in evs[i]) for i in range(args.steps)]
    attn_g_ms = [sum(e[0].elapsed_time(e[1]) for e in evs[i]) for i in range(args.steps)]
    rest_ms = [sum(e[2].elapsed_time(e[3]) for e in evs[i]) for i in range(args.steps)]
    proj_in_step_ms = float(np.mean([sum(e[2].elapsed_time(e[4]) for e in evs[i]) for i in range(args.steps)]))
    comb_wb_in_step_ms = float(np.mean([sum(e[4].elapsed_time(e[3]) for e in evs[i]) for i in range(args.steps)]))
    total_ms = float(sum(step_ms))
    total_ms_max = rkdist.max_over_ranks(total_ms, dev)
    sampler.join(timeout=2)
    clocks = sampler.summary()

    # end to end through the host-buffer entry point (H2D of the request inputs + D2H of y per step)
    # measured at N = 1 only: every rank would pin its own copy of the inputs (about 10 GB at 256K), and the
    # host-to-device copies of N ranks share the host's memory and PCIe paths, which this path does not model
    e2e = None
    if not args.no_e2e and world == 1:
        pin = lambda x: x.to("cpu").pin_memory()
        host = [(pin(wl.kv), pin(wl.q_g), pin(wl.q_l), pin(wl.z_off)) for wl, _ in layers]
        y_h = torch.empty((req.T, prof.d_model), dtype=torch.bfloat16).pin_memory()

        if n_layers > 1:      # stack entry point: inputs of layer l+1 travel while layer l computes
            bufs1 = ctx.alloc_layer_buffers(big, dev)
            ys = [y_h] + [torch.empty_like(y_h).pin_memory() for _ in range(min(n_layers, 2) - 1)]
            io = [dict(req=r, kv=h[0], q_g=h[1], q_l=h[2], z_off=h[3], W_uv=wl.w_uv, W_a=wl.w_a, W_b=wl.w_b,
                       y=ys[i % len(ys)]) for i, ((wl, r), h) in enumerate(zip(layers, host))]

        def e2e_step():
            if n_layers > 1:
                rk.rk_layer_stack_host(ctx, io, bufs, bufs1)
                return
            for (wl, r), (hk, hqg, hql, hzo) in zip(layers, host):
                ctx.rk_layer_host(r, hk, hqg, hql, hzo, wl.w_uv, wl.w_a, wl.w_b, bufs, y_h)

        e2e_step()   # warm-up
        rkdist.barrier()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(args.e2e_steps):
            e2e_step()
        torch.cuda.synchronize()
        e2e_s = (time.perf_counter() - t0)
        e2e_max = rkdist.max_over_ranks(e2e_s, dev)
        ctx.rk_poll_status()
        e2e = dict(value=rkdist.aggregate_throughput(req.T * n_layers, args.e2e_steps, world, e2e_max),
                   unit="tokens/s", h2d_bytes_per_step=int(in_bytes), d2h_bytes_per_step=int(y_h.numel() * 2 * n_layers),
                   ms_per_step=e2e_max * 1e3 / args.e2e_steps)
        del host

    # standalone HBM-bound calls (not part of the step): relocation and merge against copy bandwidth
    aux = None
    if not args.no_aux and rank == 0 and not args.value_phase:
        aux = time_stream_kernels(ctx, req, w, prof, lay, dev)
        aux.update(time_selection_rules(ctx, lay, dev))

    # where the rest of the step goes (instrumentation pass, not the timed region)
    breakdown = None
    if rank == 0:
        def ev_ms(fn):
            return timed_region(fn, stream, dev.index or 0, min_ms=150.0, lead_ms=20.0)[0]
        t_proj = ev_ms(lambda: ctx.rk_group_sliced_proj(req, bufs["O_g"], bufs["O_l"], w.w_uv, w.w_a, bufs["z_on_g"],
                                                        bufs["z_on_l"], bufs["workspace"]))
        t_comb = ev_ms(lambda: ctx.rk_combine_offline(req, bufs["z_on_g"], bufs["z_on_l"], w.z_off, None, bufs["z"]))
        t_cwb = ev_ms(lambda: ctx.rk_combine_offline(req, bufs["z_on_g"], bufs["z_on_l"], w.z_off, w.w_b, bufs["z"],
                                                     bufs["y"]))
        width = prof.n_groups * prof.o_rank
        comb_bytes = 3 * req.T * width * 2
        _, fl_proj0, fl_wb0 = algorithmic_flops(prof, req, args.value_phase)      # layer 0 alone is timed here
        breakdown = dict(sliced_proj_ms=t_proj, sliced_proj_tflops=fl_proj0 / t_proj / 1e9,
                         combine_ms=t_comb, combine_gbs=comb_bytes / t_comb / 1e6,
                         wb_gemm_ms=t_cwb - t_comb, wb_gemm_tflops=fl_wb0 / (t_cwb - t_comb) / 1e9,
                         wb_gemm_frac_of_nominal=fl_wb0 / (t_cwb - t_comb) / 1e9 / 2250.0,
                         note="each call repeated back to back for >= 150 ms (steady state under the power cap)",
                         # the same stages inside the timed steps (events between the calls; W_b = the combine + W_b call
                         # minus the stand-alone combine time), at the clock the step itself runs at
                         in_step_sliced_proj_ms=proj_in_step_ms / n_layers,
                         in_step_combine_and_wb_ms=comb_wb_in_step_ms / n_layers,
                         in_step_wb_gemm_tflops=fl_wb0 / max(comb_wb_in_step_ms / n_layers - t_comb, 1e-6) / 1e9)
        ctx.rk_poll_status()

    offline = None
    if args.with_offline and rank == 0:
        offline = time_offline_build(ctx, req, w, prof, lay, dev)

    if rank != 0:
        rkdist.shutdown()
        return

    peaks = load_peaks()
    attn_tflops = fl_attn / (np.mean(attn_ms) * 1e-3) / 1e12
    roofline = dict(bound="tensor", kernel="rk_mla_attn_kernel (Global + Local launches)" +
                                           (", output-phase instantiation, 2304 flop per pair" if args.value_phase else ""),
                    achieved=attn_tflops, peak=peaks["bf16_sustained"], unit="TFLOP/s",
                    frac=attn_tflops / peaks["bf16_sustained"], peak_source=peaks["source"] + " sustained bf16",
                    frac_of_burst=attn_tflops / peaks["bf16_burst"], frac_of_nominal=attn_tflops / 2250.0,
                    launches_per_step=2 * n_layers, ms_per_step=float(np.mean(attn_ms)),
                    ms_global_pass=float(np.mean(attn_g_ms)),
                    traffic=None if args.value_phase else (PROFILED_DRAM_TRAFFIC.get(name) or {}).get("bytes"),
                    traffic_note=(PROFILED_DRAM_TRAFFIC.get(name) or {}).get("source", "no ncu capture of this workload"),
                    traffic_captured_on=(PROFILED_DRAM_TRAFFIC.get(name) or {}).get("captured_on"),
                    tensor_pipe_use_in_cycles=None if args.value_phase else PROFILED_PIPE_USE.get(name),
                    algorithmic_dram_bytes=(PROFILED_DRAM_TRAFFIC.get(name) or {}).get("algorithmic"))
    rest_tflops = (fl_proj + fl_wb) / (np.mean(rest_ms) * 1e-3) / 1e12

    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:   # the checker is timed at N = 1 only
        run_layer(w, req)                      # leave layer 0's y in the buffer for the parity figure below
        torch.cuda.synchronize()
        rows = pick_oracle_rows(w, args.oracle_pairs)
        dt, pairs, out = oracle_sample_run(w, rows, args.value_phase)
        allp = total_pairs(prof, req)          # layer 0 (the layers have the same layout, own protected rows)
        # while the sample is at hand: parity of this very run against the checker
        from oracle.harness import rel_l2
        y_gpu = bufs["y"][torch.as_tensor(rows, device=dev)].float().cpu().numpy().astype(np.float64)
        cpu_baseline = dict(value=req.T / (dt * allp / pairs), unit="tokens/s (per layer)", cores=os.cpu_count(), kind="oracle",
                            threads=torch.get_num_threads(),
                            sample=f"{len(rows)} seeded rows, {pairs} of {allp} visible (row,key,head) pairs in "
                                   f"{dt:.1f} s, extrapolated by pair count",
                            pairs_per_s=pairs / dt, parity_rel_l2_y=rel_l2(y_gpu, out["y"]))

    line = dict(metric="mla_online_prefill_tokens_per_s_per_layer",
                value=rkdist.aggregate_throughput(req.T * n_layers, args.steps, world, total_ms_max * 1e-3),
                unit="tokens/s", n_gpus=world, steps=args.steps, warmup=args.warmup,
                ms_per_step=total_ms_max / args.steps, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype="bf16", data="synthetic",
                config=dict(workload=name, regime=args.regime, value_phase=args.value_phase, layers=n_layers, T=req.T, n_prot=req.A, n_segs=lay.n_segs,
                            heads=prof.n_heads, groups=prof.n_groups, o_rank=prof.o_rank, d_model=prof.d_model,
                            l2="inputs larger than L2" if not need_flush else "L2 flushed between iterations",
                            flops_attn=fl_attn, flops_proj=fl_proj + fl_wb),
                clocks=clocks, e2e=e2e, gpu_launches=launches_per_step * args.steps, roofline=roofline,
                proj_tflops=rest_tflops, proj_ms_per_step=float(np.mean(rest_ms)), cpu_baseline=cpu_baseline)
    if breakdown:
        line["projection_breakdown"] = breakdown
    if offline:
        line["offline_build"] = offline
    if aux:
        for k, v in aux.items():
            v["frac_of_hbm_peak"] = v["gbs"] / peaks["hbm_gbs"]
        line["hbm_kernels"] = dict(peak_gbs=peaks["hbm_gbs"], peak_source=peaks["source"] + " copy bandwidth", **aux)
    print(json.dumps(line))
    rkdist.shutdown()


if __name__ == "__main__":
    main()

#!/usr/bin/env python
"""Benchmark of the CaliDrop hot path on B200: compress-and-calibrate + calibrated decode.

One "step" is one pass of the whole hot path over one batch of synthetic input at the
32K-context configuration (batch 4, 32 query / 8 kv heads, head_dim 128, prefix 32768, window 64,
pool 7, budget 2048, 128 decode steps): the end-of-prefill compress-and-calibrate of every
layer state, then 128 calibrated decode steps over each state.  To keep the retained caches
(34 MB each) from living in the 126 MB L2 between decode steps, the step runs over
`--states` (default 8) independent layer states visited round-robin, the way the layers of a
model stack are; the prompt K/V they are compressed from alternate between `--inputs`
(default 2) independently seeded prompts of 537 MB each.

The headline `value` is the first half of the metric: achieved HBM GB/s of the decode
attention (algorithmic bytes / device time of the decode phase).  The second half,
compress+calibrate milliseconds per layer and its fraction of the tensor-core peak, is in
`compress`.  `--impl reference` times the fp64 CPU oracle instead (a deliberately slow program).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "decode attn HBM GB/s (% of peak); compress+calibrate ms/layer (% TC peak)"
UNIT = "GB/s"
FALLBACK_HBM_GBS, FALLBACK_BF16_TFLOPS = 6650.0, 1590.0
# dram__bytes_read.sum + dram__bytes_write.sum per decode launch at config 3, n_cal 64, from a one-pass
# ncu capture late in an eager sequence of launches with the caches left as the launches before it
# left them (the median launch: a sixth of the cache is still in L2; from flushed caches a launch
# reads 35.9 MB, its algorithmic bytes); reported only for that workload.
DECODE_DRAM_TRAFFIC_PER_LAUNCH = 29636608


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        d = json.load(open(path))
        return dict(hbm_gbs=float(d["hbm_gbs"]), bf16_tflops=float(d["bf16_tflops"]),
                    bf16_tflops_sustained=float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=FALLBACK_HBM_GBS, bf16_tflops=FALLBACK_BF16_TFLOPS,
                bf16_tflops_sustained=1400.0, source="fallback")


def decode_bytes(cfg, n_cal, n_kv):
    """Algorithmic bytes of one decode launch: K and V rows once for the whole query group,
    q and out, the calibration queries, one O_c row and LSE_c per head."""
    B, Hq, Hkv, D = cfg.B, cfg.Hq, cfg.Hkv, cfg.D
    return 2 * B * Hkv * n_kv * D * 2 + B * Hq * D * 2 * 2 + B * Hq * n_cal * D * 2 + B * Hq * (D * 4 + 4)


def compress_flops(cfg, n_cal):
    """Algorithmic flops of compress-and-calibrate: window scoring QK^T plus the evicted-token
    P.V (the logits of the calibration rows are already part of the scoring)."""
    E = cfg.L - cfg.budget
    return 2 * cfg.B * cfg.Hq * cfg.window * cfg.L * cfg.D + 2 * cfg.B * cfg.Hq * n_cal * E * cfg.D


def max_over_ranks(values, world, device):
    """Multi-GPU timing rule: every rank contributes its device-measured times and all of them
    continue with the maximum over the ranks (one all-reduce on the job's process group)."""
    import torch
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t.cpu()]


def whole_job_rate(units_per_rank, world, time_ms):
    """Replicas only: every rank processes the same number of units, the job's rate is all of them
    over the slowest rank's time."""
    return units_per_rank * world / (time_ms * 1e-3)


def compress_exps(cfg, n_cal, lse_supplied=False):
    """Exponentials the path evaluates per layer: one per logit in the vote pass (and in the
    statistics pass when the caller supplies no row LSE), one per (calibration row, candidate)."""
    E = cfg.L - cfg.budget
    passes = 1 if lse_supplied else 2
    return passes * cfg.B * cfg.Hq * cfg.window * cfg.L + cfg.B * cfg.Hq * n_cal * E


# special-function pipe: 16 results per clock per SM (measured with a dependent-free ex2 loop),
# 148 SMs, at the maximum SM clock
XU_PER_CLK_PER_SM, N_SMS, SM_MAX_HZ = 16, 148, 1.965e9


def compress_bytes(cfg):
    """Minimum bytes: K once, V once, the gather's read and write of the kept rows."""
    kv = cfg.B * cfg.Hkv * cfg.L * cfg.D * 2
    return 2 * kv + 4 * cfg.B * cfg.Hkv * cfg.budget * cfg.D * 2


def compress_floors(cfg, n_cal, lse_supplied, peaks):
    """Microseconds per layer that each of the three co-limiting resources needs on its own."""
    return {"tensor": compress_flops(cfg, n_cal) / (peaks["bf16_tflops_sustained"] * 1e12) * 1e6,
            "hbm": compress_bytes(cfg) / (peaks["hbm_gbs"] * 1e9) * 1e6,
            "exp": compress_exps(cfg, n_cal, lse_supplied) / (XU_PER_CLK_PER_SM * N_SMS * SM_MAX_HZ) * 1e6}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu_index, self.rows, self.proc = gpu_index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                 "-i", str(self.gpu_index)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for r in self.rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1])); mx.append(float(r[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"),
                               r[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


# ------------------------------------------------------------------------------------ GPU arm
def run_gpu(args):
    import torch
    import torch.distributed as dist

    from paper_2507_19906_b200 import binding as cd
    from paper_2507_19906_b200 import workload as wl

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    cd.load()  # fails loudly if the CUDA library is missing: there is no fallback
    peaks = load_peaks()

    cfg = wl.CONFIGS[args.config]
    # every rank is an independent replica with its own seeds (the path has no exchange step)
    cfg = cfg.scaled(seed=cfg.seed + 7919 * rank)
    n_cal = cfg.window if args.n_cal is None else args.n_cal
    T = cfg.steps if args.decode_steps is None else args.decode_steps
    S, NI = args.states, args.inputs
    cap = cfg.budget + T
    p = cd.make_params(B=cfg.B, Hq=cfg.Hq, Hkv=cfg.Hkv, L=cfg.L, window=cfg.window, pool=cfg.pool,
                       budget=cfg.budget, n_cal=n_cal, cap=cap, theta1=0.7, theta2=0.85)

    def dev_bf16(bits):
        return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)

    def pin(bits):
        return torch.from_numpy(bits.view(np.int16)).pin_memory()

    t_gen = time.time()
    inputs, host_inputs = [], []
    for i in range(NI):
        c = cfg.scaled(seed=cfg.seed + 101 * i)
        Qb = wl.gen_q_obs(c)
        Kb, Vb = wl.gen_kv(c)
        inputs.append((dev_bf16(Qb), dev_bf16(Kb), dev_bf16(Vb)))
        if args.e2e_steps > 0:
            host_inputs.append((pin(Qb), pin(Kb), pin(Vb)))
        if i == 0:
            q_bits, kn_bits, vn_bits = wl.gen_decode_inputs(c, Qb, steps=T)
            sample_inputs = (c, Qb, Kb, Vb)
    dq, dkn, dvn = dev_bf16(q_bits), dev_bf16(kn_bits), dev_bf16(vn_bits)
    hq_, hkn, hvn = pin(q_bits), pin(kn_bits), pin(vn_bits)
    t_gen = time.time() - t_gen

    states = [cd.alloc_layer_state(p) for _ in range(S)]
    outs = [torch.empty((cfg.B, cfg.Hq, cfg.D), dtype=torch.bfloat16, device="cuda") for _ in range(S)]
    lses = [torch.empty((cfg.B, cfg.Hq), dtype=torch.float32, device="cuda") for _ in range(S)]
    flgs = [torch.empty((cfg.B, cfg.Hq), dtype=torch.uint8, device="cuda") for _ in range(S)]

    lse_in = [None] * NI
    if args.lse_obs:
        # what a prefill attention kernel would hand over: here taken from an untimed compress call
        lay = cd.calidrop_compress_workspace_layout(p)
        n_lse = cfg.B * cfg.Hq * cfg.window
        for i in range(NI):
            Qd, Kd, Vd = inputs[i]
            st = states[0]
            cd.calidrop_compress(p, Qd, Kd, Vd, None, st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c,
                                 st.C_q, st.ws_compress)
            torch.cuda.synchronize()
            lse_in[i] = st.ws_compress[lay.row_lse_offset:lay.row_lse_offset + 4 * n_lse].view(torch.float32).clone()

    def compress_phase():
        for s, st in enumerate(states):
            Qd, Kd, Vd = inputs[s % NI]
            cd.calidrop_compress(p, Qd, Kd, Vd, lse_in[s % NI], st.kept_idx, st.K_kept, st.V_kept, st.O_c,
                                 st.LSE_c, st.C_q, st.ws_compress)

    if args.batched_decode:
        # one launch per decode step covering all layer states (calidrop_decode_batched)
        ws_b = torch.zeros((cd.calidrop_decode_workspace_bytes(p, cap) * S,), dtype=torch.uint8, device="cuda")
        layer_arrays = [cd.make_decode_layers([
            dict(q=dq[t], k_new=dkn[t], v_new=dvn[t], K_kept=st.K_kept, V_kept=st.V_kept, O_c=st.O_c,
                 LSE_c=st.LSE_c, C_q=st.C_q, out=outs[s], lse_out=lses[s], flags=flgs[s])
            for s, st in enumerate(states)]) for t in range(T)]

    def decode_phase():
        if args.batched_decode:
            for t in range(T):
                cd.calidrop_decode_batched(p, layer_arrays[t], cfg.budget + t, ws_b)
            return
        for t in range(T):
            for s, st in enumerate(states):
                cd.calidrop_decode(p, dq[t], dkn[t], dvn[t], st.K_kept, st.V_kept, cfg.budget + t, st.O_c,
                                   st.LSE_c, st.C_q, outs[s], lses[s], flgs[s], st.ws_decode)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
            torch.cuda.synchronize()

    for w in range(max(1, args.warmup - 2) if not args.no_graph else args.warmup):
        l0 = cd.calidrop_launch_count()
        compress_phase()
        decode_phase()
        launches_per_step = cd.calidrop_launch_count() - l0
    barrier()
    run_compress, run_decode = compress_phase, decode_phase
    if not args.no_graph:
        # The launch sequence of a step is fixed, so it is captured once into two CUDA graphs
        # (the library launches on the capturing stream like on any other) and replayed.
        g_comp, g_dec = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_comp):
            compress_phase()
        with torch.cuda.graph(g_dec):
            decode_phase()
        run_compress, run_decode = g_comp.replay, g_dec.replay
        for _ in range(2):
            run_compress()
            run_decode()
        barrier()

    sampler = ClockSampler(local)
    sampler.start()
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    launches0 = cd.calidrop_launch_count()
    barrier()
    for k in range(args.steps):
        ev[k][0].record()
        run_compress()
        ev[k][1].record()
        run_decode()
        ev[k][2].record()
    barrier()
    launches = cd.calidrop_launch_count() - launches0
    if not args.no_graph:
        launches = args.steps * launches_per_step
    clocks = sampler.stop()
    t_comp = sum(e[0].elapsed_time(e[1]) for e in ev)   # ms over all timed steps
    t_dec = sum(e[1].elapsed_time(e[2]) for e in ev)
    t_tot = sum(e[0].elapsed_time(e[2]) for e in ev)
    t_comp, t_dec, t_tot = max_over_ranks([t_comp, t_dec, t_tot], world, "cuda")
    dec_step_ms = sorted(e[1].elapsed_time(e[2]) for e in ev)      # this rank's timed repetitions of the decode phase
    comp_step_ms = sorted(e[0].elapsed_time(e[1]) for e in ev)

    dec_bytes_step = sum(decode_bytes(cfg, n_cal, cfg.budget + t + 1) for t in range(T)) * S
    dec_launches = T * (1 if args.batched_decode else S) * args.steps
    dec_gbs = dec_bytes_step * args.steps / (t_dec * 1e-3) / 1e9
    comp_ms_layer = t_comp / (args.steps * S)
    comp_tflops = compress_flops(cfg, n_cal) / (comp_ms_layer * 1e-3) / 1e12
    comp_gbs = compress_bytes(cfg) / (comp_ms_layer * 1e-3) / 1e9

    # ---------------- end to end through the host-buffer entry points (copies inside the timed region)
    e2e = None
    if args.e2e_steps > 0:
        Qd, Kd, Vd = inputs[0]
        n_kept = min(cfg.budget, cfg.L)
        kept_h = torch.empty((cfg.B, cfg.Hkv, n_kept), dtype=torch.int32).pin_memory()
        Oc_h = torch.empty((cfg.B, cfg.Hq, n_cal, cfg.D), dtype=torch.float32).pin_memory()
        Lc_h = torch.empty((cfg.B, cfg.Hq, n_cal), dtype=torch.float32).pin_memory()
        out_h = torch.empty((cfg.B, cfg.Hq, cfg.D), dtype=torch.bfloat16).pin_memory()
        dq1 = torch.empty_like(dq[0]); dk1 = torch.empty_like(dkn[0]); dv1 = torch.empty_like(dvn[0])

        def e2e_step():
            for s, st in enumerate(states):
                Qh, Kh, Vh = host_inputs[s % NI]
                cd.calidrop_compress_host(p, Qh, Kh, Vh, None, kept_h, Oc_h, Lc_h, Qd, Kd, Vd, None,
                                          st.kept_idx, st.K_kept, st.V_kept, st.O_c, st.LSE_c, st.C_q,
                                          st.ws_compress)
            for t in range(T):
                for s, st in enumerate(states):
                    cd.calidrop_decode_host(p, hq_[t], hkn[t], hvn[t], out_h, None, None, dq1, dk1, dv1,
                                            st.K_kept, st.V_kept, cfg.budget + t, st.O_c, st.LSE_c, st.C_q,
                                            outs[s], None, None, st.ws_decode)

        e2e_step()
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        e1.record()
        barrier()
        tot_ms = e0.elapsed_time(e1)
        tot_ms = max_over_ranks([tot_ms], world, "cuda")[0]
        h2d = S * (cfg.B * cfg.Hq * cfg.window * cfg.D * 2 + 2 * cfg.B * cfg.Hkv * cfg.L * cfg.D * 2) + \
            T * S * (cfg.B * cfg.Hq * cfg.D * 2 + 2 * cfg.B * cfg.Hkv * cfg.D * 2)
        d2h = S * (kept_h.numel() * 4 + Oc_h.numel() * 4 + Lc_h.numel() * 4) + T * S * out_h.numel() * 2
        e2e = {"value": whole_job_rate(dec_bytes_step * args.e2e_steps, world, tot_ms) / 1e9, "unit": UNIT,
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
               "ms_per_step": tot_ms / args.e2e_steps,
               "note": "decode algorithmic bytes / whole end-to-end step time (host copies of the prompt "
                       "K/V, compress, and every decode step's host round trip included)"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---------------- the recompute branch, as an extra (not part of the step)
    recompute = None
    if args.recompute and cfg.budget < cfg.L:
        st = states[0]
        Qd, Kd, Vd = inputs[0]
        n_e = cfg.L - cfg.budget
        ev_idx = torch.empty((cfg.B, cfg.Hkv, n_e), dtype=torch.int32, device="cuda")
        K_e = torch.empty((cfg.B, cfg.Hkv, n_e, cfg.D), dtype=torch.bfloat16, device="cuda")
        V_e = torch.empty_like(K_e)
        reps = 10
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        for it in range(2):   # the first round warms up
            torch.cuda.synchronize()
            evs[0].record()
            cd.calidrop_gather_evicted(p, Kd, Vd, st.kept_idx, ev_idx, K_e, V_e, st.ws_compress)
            evs[1].record()
            for r in range(reps):
                cd.calidrop_recalibrate(p, dq[r % T], K_e, V_e, n_e, r % n_cal, st.O_c, st.LSE_c, st.C_q, st.ws_decode)
            evs[2].record()
            torch.cuda.synchronize()
        ev_bytes = 2 * cfg.B * cfg.Hkv * n_e * cfg.D * 2
        t_g, t_r = evs[0].elapsed_time(evs[1]), evs[1].elapsed_time(evs[2]) / reps
        # offload to and reload from page-locked host memory on a copy stream (Algorithm 1 line 4,
        # Algorithm 2 line 4), alone and with decode steps running on the compute stream
        K_h = torch.empty(K_e.shape, dtype=torch.bfloat16).pin_memory()
        V_h = torch.empty(V_e.shape, dtype=torch.bfloat16).pin_memory()
        side = torch.cuda.Stream()
        c0, c1, c2 = (torch.cuda.Event(enable_timing=True) for _ in range(3))
        for it in range(2):
            torch.cuda.synchronize()
            c0.record(side)
            cd.calidrop_offload_evicted(p, n_e, K_e, V_e, K_h, V_h, side)
            c1.record(side)
            cd.calidrop_reload_evicted(p, n_e, K_h, V_h, K_e, V_e, side)
            c2.record(side)
            torch.cuda.synchronize()
        t_off, t_rel = c0.elapsed_time(c1), c1.elapsed_time(c2)
        n_dec = min(T, 32)

        def some_decode_steps():
            for t in range(n_dec):
                for s_, st_ in enumerate(states):
                    cd.calidrop_decode(p, dq[t], None, None, st_.K_kept, st_.V_kept, cfg.budget, st_.O_c, st_.LSE_c,
                                       st_.C_q, outs[s_], lses[s_], flgs[s_], st_.ws_decode)

        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        some_decode_steps()
        torch.cuda.synchronize()
        d0.record(); some_decode_steps(); d1.record()
        torch.cuda.synchronize()
        t_dec_alone = d0.elapsed_time(d1)
        c0.record(side)
        cd.calidrop_reload_evicted(p, n_e, K_h, V_h, K_e, V_e, side)
        c1.record(side)
        d0.record(); some_decode_steps(); d1.record()
        torch.cuda.synchronize()
        t_dec_busy, t_rel_busy = d0.elapsed_time(d1), c0.elapsed_time(c1)
        recompute = {"n_evict": n_e, "gather_evicted_ms": t_g,
                     "offload_ms": t_off, "offload_gbs": ev_bytes / (t_off * 1e-3) / 1e9,
                     "reload_ms": t_rel, "reload_gbs": ev_bytes / (t_rel * 1e-3) / 1e9,
                     "reload_beside_decode": {
                         "decode_launches": n_dec * S, "decode_ms_alone": t_dec_alone, "decode_ms_with_reload": t_dec_busy,
                         "reload_ms_with_decode": t_rel_busy,
                         "note": "eager decode launches on the compute stream while the reload runs on a copy stream"},
                     "gather_evicted_gbs": 2 * ev_bytes / (t_g * 1e-3) / 1e9,     # rows read and written
                     "recalibrate_us": t_r * 1e3, "recalibrate_gbs": ev_bytes / (t_r * 1e-3) / 1e9,
                     "recalibrate_frac_of_measured_hbm": ev_bytes / (t_r * 1e-3) / 1e9 / peaks["hbm_gbs"]}

    # ---------------- the oracle beside it (rank 0, bounded sample)
    cpu = None
    if not args.no_cpu_baseline and world == 1:
        cpu = time_oracle(sample_inputs, n_cal, T, q_bits, kn_bits, vn_bits, args.cpu_units)

    avg_launch_s = t_dec * 1e-3 / dec_launches
    bytes_per_launch = dec_bytes_step / (T * (1 if args.batched_decode else S))
    result = {
        "metric": METRIC, "value": whole_job_rate(dec_bytes_step * args.steps, world, t_dec) / 1e9, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": t_tot / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"config {args.config}: B{cfg.B} {cfg.Hq}q/{cfg.Hkv}kv D128 prefix {cfg.L} "
                               f"window {cfg.window} pool {cfg.pool} budget {cfg.budget} n_cal {n_cal} "
                               f"{T} decode steps",
                   "layer_states": S, "prompt_inputs": NI,
                   "l2": f"inputs larger than L2: {S} retained caches ({S * bytes_per_launch / 1e6:.0f} MB) "
                         f"visited round-robin, prompts of {2 * cfg.B * cfg.Hkv * cfg.L * cfg.D * 2 / 1e6:.0f} MB",
                   "lse_obs": "supplied by the caller (statistics pass skipped)" if args.lse_obs
                   else "not supplied (row statistics recomputed inside the step)",
                   "launch": "eager C-ABI calls" if args.no_graph else "CUDA-graph replay of the captured C-ABI calls",
                   "decode_entry": "calidrop_decode_batched over the layer states" if args.batched_decode
                   else "calidrop_decode per layer state",
                   "parallelism": "replicas only" if world > 1 else "single GPU"},
        "decode": {"us_per_launch": avg_launch_s * 1e6, "gbs": dec_gbs, "launches": dec_launches,
                   "bytes_per_launch": bytes_per_launch,
                   # spread over the timed repetitions of the decode phase (each T x states launches)
                   "us_per_launch_median": dec_step_ms[len(dec_step_ms) // 2] * 1e3 / (dec_launches / args.steps),
                   "us_per_launch_min": dec_step_ms[0] * 1e3 / (dec_launches / args.steps),
                   "us_per_launch_max": dec_step_ms[-1] * 1e3 / (dec_launches / args.steps),
                   "repetitions": args.steps,
                   "frac_of_measured_hbm": dec_gbs / peaks["hbm_gbs"], "frac_of_nominal_8tbs": dec_gbs / 8000.0},
        "compress": {"ms_per_layer": comp_ms_layer,
                     "ms_per_layer_median": comp_step_ms[len(comp_step_ms) // 2] / S,
                     # the three floors of the step (tensor pipe at the sustained bf16 peak, copy bandwidth on
                     # the minimum bytes, special-function pipe on the exponentials); the step is bound by
                     # the largest, and frac_of_bound = that floor / measured time
                     "floor_us": compress_floors(cfg, n_cal, args.lse_obs, peaks),
                     "frac_of_bound": max(compress_floors(cfg, n_cal, args.lse_obs, peaks).values())
                     / (comp_ms_layer * 1e3),
                     "algorithmic_tflops": comp_tflops,
                     "frac_of_bf16_peak_burst": comp_tflops / peaks["bf16_tflops"],
                     "frac_of_bf16_peak_sustained": comp_tflops / peaks["bf16_tflops_sustained"],
                     "min_bytes_gbs": comp_gbs, "frac_of_measured_hbm": comp_gbs / peaks["hbm_gbs"],
                     "exp_per_s": compress_exps(cfg, n_cal, args.lse_obs) / (comp_ms_layer * 1e-3),
                     "frac_of_xu_peak": compress_exps(cfg, n_cal, args.lse_obs) / (comp_ms_layer * 1e-3)
                     / (XU_PER_CLK_PER_SM * N_SMS * SM_MAX_HZ)},
        "roofline": {"bound": "hbm", "kernel": "decode_kernel", "achieved": dec_gbs, "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": dec_gbs / peaks["hbm_gbs"], "peak_source": peaks["source"],
                     "traffic": DECODE_DRAM_TRAFFIC_PER_LAUNCH
                     if (args.config == 3 and n_cal == 64 and not args.batched_decode) else None,
                     "traffic_state": "steady state of the eager launch sequence (caches not flushed)"},
        "roofline_compress": {"bound": "tensor", "achieved": comp_tflops, "peak": peaks["bf16_tflops_sustained"],
                              "unit": "TFLOP/s", "frac": comp_tflops / peaks["bf16_tflops_sustained"],
                              "peak_source": peaks["source"] + " (sustained bf16 GEMM)"},
        "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks,
        "recompute": recompute, "input_generation_s": t_gen,
    }
    print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def time_oracle(sample_inputs, n_cal, T, q_bits, kn_bits, vn_bits, n_units):
    """Time the fp64 oracle, as it stands, on a bounded sample of the same workload."""
    import oracle
    cfg, Qb, Kb, Vb = sample_inputs
    G = cfg.G
    n_units = min(n_units, cfg.Hkv)
    Qs = np.ascontiguousarray(Qb[:1, : n_units * G])
    Ks, Vs = np.ascontiguousarray(Kb[:1, :n_units]), np.ascontiguousarray(Vb[:1, :n_units])
    t0 = time.time()
    r = oracle.compress(Qs, Ks, Vs, window=cfg.window, pool=cfg.pool, budget=cfg.budget, n_cal=n_cal,
                        cap=cfg.budget + T)
    t_comp = time.time() - t0
    steps = min(T, 4)
    t0 = time.time()
    for t in range(steps):
        oracle.decode(np.ascontiguousarray(q_bits[t, :1, : n_units * G]),
                      np.ascontiguousarray(kn_bits[t, :1, :n_units]),
                      np.ascontiguousarray(vn_bits[t, :1, :n_units]), r.K_kept, r.V_kept, cfg.budget + t,
                      r.O_c, r.LSE_c, r.C_q)
    t_dec = (time.time() - t0) / steps
    frac = n_units / (cfg.B * cfg.Hkv)
    sub = cfg.scaled(B=1, Hq=n_units * G, Hkv=n_units)
    dec_b = np.mean([decode_bytes(sub, n_cal, cfg.budget + t + 1) for t in range(steps)])
    return {"value": dec_b / t_dec / 1e9, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
            "sample": f"{n_units} of {cfg.B * cfg.Hkv} (batch, kv-head) units: compress-and-calibrate once, "
                      f"{steps} decode steps",
            "compress_ms_per_layer_extrapolated": t_comp * 1e3 / frac,
            "decode_us_per_step_extrapolated": t_dec * 1e6 / frac,
            "host_cores": os.cpu_count()}


# ------------------------------------------------------------------------------ reference arm
def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from paper_2507_19906_b200 import workload as wl
    cfg = wl.CONFIGS[args.config]
    n_cal = cfg.window if args.n_cal is None else args.n_cal
    T = cfg.steps if args.decode_steps is None else args.decode_steps
    n_units = min(args.cpu_units, cfg.Hkv)
    G = cfg.G
    Qb = wl.gen_q_obs(cfg)[:1, : n_units * G]
    units = [wl.gen_kv_unit(cfg, 0, 0, h) for h in range(n_units)]
    Ks = np.ascontiguousarray(np.stack([u[0] for u in units])[None])
    Vs = np.ascontiguousarray(np.stack([u[1] for u in units])[None])
    Qs = np.ascontiguousarray(Qb)
    q_bits, kn_bits, vn_bits = wl.gen_decode_inputs(cfg, wl.gen_q_obs(cfg), steps=T)
    dsteps = min(T, 4)
    sub = cfg.scaled(B=1, Hq=n_units * G, Hkv=n_units)

    def one_step():
        t0 = time.time()
        r = oracle.compress(Qs, Ks, Vs, window=cfg.window, pool=cfg.pool, budget=cfg.budget, n_cal=n_cal,
                            cap=cfg.budget + T)
        t1 = time.time()
        for t in range(dsteps):
            oracle.decode(np.ascontiguousarray(q_bits[t, :1, : n_units * G]),
                          np.ascontiguousarray(kn_bits[t, :1, :n_units]),
                          np.ascontiguousarray(vn_bits[t, :1, :n_units]), r.K_kept, r.V_kept, cfg.budget + t,
                          r.O_c, r.LSE_c, r.C_q)
        t2 = time.time()
        return t1 - t0, t2 - t1

    for _ in range(args.warmup):
        one_step()
    tc = td = 0.0
    for _ in range(args.steps):
        a, b = one_step()
        tc += a; td += b
    dec_b = sum(decode_bytes(sub, n_cal, cfg.budget + t + 1) for t in range(dsteps))
    value = dec_b * args.steps / td / 1e9
    frac = n_units / (cfg.B * cfg.Hkv)
    sample = (f"{n_units} of {cfg.B * cfg.Hkv} (batch, kv-head) units per step: compress-and-calibrate once, "
              f"{dsteps} of {T} decode steps")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": (tc + td) * 1e3 / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"config {args.config}: B{cfg.B} {cfg.Hq}q/{cfg.Hkv}kv D128 prefix {cfg.L} "
                               f"window {cfg.window} pool {cfg.pool} budget {cfg.budget} n_cal {n_cal} "
                               f"{T} decode steps", "sample": sample},
        "compress_ms_per_layer_extrapolated": tc * 1e3 / args.steps / frac,
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.max_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def replica_command(n_gpus, argv, port):
    """The command line that runs this file as n_gpus processes on this node, one rank per GPU."""
    return [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n_gpus}",
            "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)


def spawn_replicas(n_gpus, argv, run=None):
    """`bench.py --gpus N` without a launcher: start the N replicas (the path has no exchange step, so
    the ranks only meet in the barrier and the max-over-ranks of the timing) and pass their output on."""
    port = 29500 + os.getpid() % 1000
    return (run or subprocess.call)(replica_command(n_gpus, argv, port))


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=3)
    ap.add_argument("--n-cal", type=int, default=None, help="calibration rows (default: the window)")
    ap.add_argument("--decode-steps", type=int, default=None)
    ap.add_argument("--states", type=int, default=8, help="independent layer states visited round-robin")
    ap.add_argument("--inputs", type=int, default=2, help="independently seeded prompts")
    ap.add_argument("--e2e-steps", type=int, default=1)
    ap.add_argument("--cpu-units", type=int, default=4)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batched-decode", action="store_true",
                    help="one calidrop_decode_batched launch per decode step over all layer states")
    ap.add_argument("--recompute", action="store_true",
                    help="also time calidrop_gather_evicted and calidrop_recalibrate (the recompute branch of "
                         "Algorithm 2) on the first layer state, outside the timed step; reported under 'recompute'")
    ap.add_argument("--lse-obs", action="store_true",
                    help="supply the row log-sum-exp of the prefill attention to calidrop_compress (as a prefill "
                         "kernel would), so the statistics pass is skipped; not the default workload")
    ap.add_argument("--no-graph", action="store_true", help="launch every call eagerly instead of replaying CUDA graphs")
    args = ap.parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started as a plain process: become the launcher of N replica processes, one per GPU
        return spawn_replicas(args.gpus, sys.argv[1:] if argv is None else list(argv))
    if args.impl == "reference":
        run_reference(args)
    else:
        run_gpu(args)
    return 0


if __name__ == "__main__":
    sys.exit(main())

#!/usr/bin/env python
"""Benchmark of the HEART layer-step (drift + mask prediction + block-sparse attention) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload hunyuan-720p] [--impl reference]

A "step" is one heart_step call = one whole pass of the hot path over one denoising step of
synthetic Q/K/V (seeded, shaped like the paper's Wan2.1 / HunyuanVideo activations), with the TMR
state carried from step to step so refresh and reuse mix as in a real sweep.  Prints ONE JSON line.

The headline workload is the largest single-GPU configuration (hunyuan-720p: 24 heads, 118 800
tokens, block 128, every head refreshing at every step); the other four configurations are measured
in the same run on a few steps each and reported in `per_workload`, each with its own clock record.

The path does not shard (one layer's heads could be split across GPUs with no exchange, but the
library is a single-GPU kernel library): with --gpus N every rank runs an independent replica
("replicas only"), and `value` is the time per layer-step of the whole job = max-over-ranks step
time / N.  Run without torchrun, --gpus N starts the N ranks itself.

--impl reference times the CPU oracle (oracle/) as it stands on the host cores, on a bounded
sample of the same workload, and prints the same line with "impl": "reference".
"""
import argparse
import json
import os
import socket
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "ms per layer-step (drift+mask+attn)"
HEADLINE = "hunyuan-720p"
OTHERS = ("tiny", "wan1.3b-480p", "wan14b-480p", "wan14b-720p")
TRAFFIC_TABLE = os.path.join(ROOT, "profiles", "attn_tc_kernel_dram_traffic.txt")


def parse():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--workload", default=HEADLINE)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--cpu-sample-rows", type=int, default=0,
                    help="query blocks the CPU oracle attends per step (0: sized for about a second per step)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-per-workload", action="store_true", help="measure the headline workload only")
    return ap.parse_args()


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm_gbs": d["hbm_gbs"], "bf16_tflops": d["bf16_tflops"],
                "bf16_tflops_sustained": d.get("bf16_tflops_sustained", d["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def dram_traffic(workload):
    """DRAM bytes per attention launch (ncu, dram__bytes_read.sum + dram__bytes_write.sum) from the table
    under profiles/ that the captures are summarised into; None where no capture exists."""
    try:
        for line in open(TRAFFIC_TABLE):
            f = line.split()
            if len(f) >= 2 and not line.startswith("#") and f[0] == workload:
                return float(f[1])
    except OSError:
        pass
    return None


def config_of(wl):
    """The workload description both arms print (identical in both)."""
    return {"workload": wl.name, "B": wl.B, "H": wl.H, "N": wl.N, "grid": list(wl.grid), "D": wl.D,
            "block": wl.block, "n_blocks": wl.n_blocks, "pos_scale": float(wl.pos_scale[0]), "seed": wl.seed}


class ClockSampler:
    """SM clock and throttle reasons of one GPU, read (never set) through NVML every few milliseconds
    in a background thread while the timed region runs; `nvidia-smi -lms` is the fallback."""

    REASONS = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20, "sw_power_cap": 0x4}
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid, period_s=0.004):
        import threading

        self.sm, self.mx, self.reasons, self.p, self.thread = [], [], set(), None, None
        self.stop_flag = threading.Event()
        try:
            import pynvml

            pynvml.nvmlInit()
            try:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            mx = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))

            def loop():
                while not self.stop_flag.is_set():
                    try:
                        self.sm.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
                        self.mx.append(mx)
                        bits = int(pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h))
                        for name, bit in self.REASONS.items():
                            if bits & bit:
                                self.reasons.add(name)
                    except Exception:
                        pass
                    time.sleep(period_s)

            self.thread = threading.Thread(target=loop, daemon=True)
            self.thread.start()
            self.how = "nvml"
        except Exception:
            self.how = "nvidia-smi"
            self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            try:
                self.p = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.FIELDS}",
                                           "--format=csv,noheader,nounits", "-lms", "50"],
                                          stdout=self.f, stderr=subprocess.DEVNULL)
            except OSError:
                self.how = "unavailable"

    def stop(self):
        if self.thread is not None:
            self.stop_flag.set()
            self.thread.join()
        elif self.p is not None:
            time.sleep(0.1)
            self.p.terminate()
            self.p.wait()
            self.f.flush()
            for l in open(self.f.name):
                r = l.strip().split(", ")
                try:
                    self.sm.append(float(r[0]))
                    self.mx.append(float(r[1]))
                except (ValueError, IndexError):
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[4:8]):
                    if v.strip().lower().startswith("active"):
                        self.reasons.add(name)
            os.unlink(self.f.name)
        return {"sm_mhz": statistics.median(self.sm) if self.sm else None,
                "sm_max_mhz": max(self.mx) if self.mx else None, "samples": len(self.sm),
                "reasons": sorted(self.reasons), "source": self.how}


def retained_flops(torch, st, wl):
    """4 * (real query rows) * (real key rows) * D summed over the retained pairs (never padding).
    Returns device scalars (flops, pairs): no host synchronisation."""
    nb, b, N = wl.n_blocks, wl.block, wl.N
    last = N - (nb - 1) * b
    cnt = st.kv_cnt.to(torch.float64)                                    # [R, nb]
    has_last = ((st.mask_bits[:, :, (nb - 1) // 32] >> ((nb - 1) % 32)) & 1).to(torch.float64)
    keys = cnt * b - has_last * (b - last)                               # real key rows per query block
    qrows = torch.full((nb,), float(b), dtype=torch.float64, device=cnt.device)
    qrows[nb - 1] = last
    return 4.0 * wl.D * (keys * qrows[None, :]).sum(), cnt.sum()


def attention_roofline(pk, tflops, clocks, region_ms, flops_step, ms_attn, traffic):
    """The attention fraction against both measured cuBLAS peaks, and which of the two applies to this
    run: the sustained one when the clock record shows the power cap (or the timed region lasted
    seconds), the burst one when the SM clock sat at its maximum for a region of milliseconds."""
    capped = bool(clocks) and "sw_power_cap" in (clocks.get("reasons") or [])
    long_region = region_ms >= 1000.0
    which = "sustained" if (capped or long_region) else "burst"
    peak = pk["bf16_tflops_sustained"] if which == "sustained" else pk["bf16_tflops"]
    why = ("sw_power_cap active during the timed passes" if capped else
           "timed region of %.0f ms" % region_ms if long_region else
           "SM clock at its maximum with no throttle reason, region of %.0f ms" % region_ms)
    return {"kernel": "block-sparse attention", "bound": "tensor", "achieved": tflops, "peak": peak,
            "unit": "TFLOP/s", "frac": tflops / peak, "traffic": traffic,
            "peak_source": f"{pk['source']} cuBLAS bf16, {which} figure ({why})",
            "frac_of_burst_peak": tflops / pk["bf16_tflops"], "burst_peak": pk["bf16_tflops"],
            "frac_of_sustained_peak": tflops / pk["bf16_tflops_sustained"],
            "sustained_peak": pk["bf16_tflops_sustained"],
            "arithmetic": "%.4g flop per launch / %.4f ms = %.1f TFLOP/s; / %.1f = %.3f" % (
                flops_step, ms_attn, tflops, peak, tflops / peak),
            "flops_per_launch": flops_step, "ms_per_launch": ms_attn}


def measure(torch, heart, inputs, replicas, wl, K, W, dev, pk, rank, sampler_uuid, full):
    """W warm-up + K timed heart_step calls on device-resident inputs, then the per-stage, accounting,
    back-to-back and (where it fits in time) dense passes.  Returns (record, context for e2e/cpu)."""
    # every step reads its own Q/K/V tensors, all resident before anything is timed; if K + W steps would not
    # fit in ~100 GB the steps cycle through as many sets as do (still never the tensors of the step before)
    step_bytes = 3 * 2 * wl.R * wl.N * wl.D
    n_inputs = max(2, min(K + W, int(100e9 // step_bytes)))
    seq = inputs.Sequence(wl, dev)
    pool = []
    for t in range(n_inputs):
        pool.append(seq.bf16())
        if t + 1 < n_inputs:
            seq.advance()
    del seq
    steps_in = [pool[t % n_inputs] for t in range(K + W)]
    cfg = heart.make_config(wl.B, wl.H, wl.N, wl.block)
    st, ws = heart.State(cfg, dev), heart.new_workspace(cfg, dev)
    delta = torch.tensor(wl.delta, dtype=torch.float64, device=dev)
    tau = torch.tensor(wl.tau, dtype=torch.float64, device=dev)
    O = torch.empty_like(steps_in[0][0])
    drift = torch.empty(wl.R, dtype=torch.float64, device=dev)
    refresh = torch.empty(wl.R, dtype=torch.uint8, device=dev)

    def step(t):
        Q, Kt, V = steps_in[t]
        heart.heart_step(cfg, Q, Kt, V, delta, tau, st, O, ws, drift_out=drift, refresh_out=refresh)

    def barrier():
        replicas.barrier()
        torch.cuda.synchronize()

    for t in range(W):
        step(t)
    torch.cuda.synchronize()
    ckpt = st.state_dict()  # state after warm-up: the later passes restart from here

    # ---- timed region: exactly K steps, device-resident inputs
    sampler = ClockSampler(sampler_uuid) if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches = 0
    barrier()
    t_wall = time.perf_counter()
    e0.record()
    for k in range(K):
        step(W + k)
        launches += heart.heart_last_launch_count()
    e1.record()
    barrier()
    wall_ms = (time.perf_counter() - t_wall) * 1e3
    clocks = sampler.stop() if sampler else None
    total_ms = e0.elapsed_time(e1)
    assert heart.heart_get_status(ws) == 0
    total_ms = replicas.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / K

    # ---- per-stage pass: the same K steps as three C-ABI calls, one event pair per call.  Nothing here
    # synchronises with the host, and nothing but the three calls and the event records is enqueued.  The
    # mask call reuses the block means that the drift call has just left in the workspace.
    st.load_state_dict(ckpt)
    stage_ev = []
    r2 = torch.empty_like(refresh)
    torch.cuda.synchronize()
    sampler2 = ClockSampler(sampler_uuid) if rank == 0 else None  # this pass has its own clock record
    for k in range(K):
        Q, Kt, V = steps_in[W + k]
        e = [torch.cuda.Event(enable_timing=True) for _ in range(4)]
        e[0].record()
        heart.heart_drift(cfg, Q, Kt, delta, st, ws, refresh_out=r2)
        e[1].record()
        heart.heart_predict_mask(cfg, Q, Kt, tau, st, ws, refresh=r2, means_valid=True)
        e[2].record()
        heart.heart_block_sparse_attn(cfg, Q, Kt, V, st.kv_idx, st.kv_cnt, O, ws)
        e[3].record()
        stage_ev.append(e)
    torch.cuda.synchronize()
    clocks_stage = sampler2.stop() if sampler2 else None
    assert heart.heart_get_status(ws) == 0
    # ---- accounting pass (untimed): the same decisions and masks again from the same state; the flop /
    # pair / refresh counts are accumulated on the device.
    st.load_state_dict(ckpt)
    acc = torch.zeros(3, dtype=torch.float64, device=dev)  # retained flops, retained pairs, refreshed heads
    for k in range(K):
        Q, Kt, V = steps_in[W + k]
        heart.heart_drift(cfg, Q, Kt, delta, st, ws, refresh_out=r2)
        heart.heart_predict_mask(cfg, Q, Kt, tau, st, ws, refresh=r2, means_valid=True)
        f, p = retained_flops(torch, st, wl)
        acc += torch.stack([f, p, r2.sum().to(torch.float64)])
    torch.cuda.synchronize()
    flops_total, pairs_total, refreshed = (float(x) for x in acc.tolist())
    ms_drift = sum(e[0].elapsed_time(e[1]) for e in stage_ev) / K
    ms_mask = sum(e[1].elapsed_time(e[2]) for e in stage_ev) / K
    ms_attn = sum(e[2].elapsed_time(e[3]) for e in stage_ev) / K
    flops_step = flops_total / K
    density = pairs_total / K / (wl.R * wl.n_blocks ** 2)
    dense_flops = 4.0 * wl.R * float(wl.N) ** 2 * wl.D
    attn_tflops = flops_step / (ms_attn * 1e-3) / 1e12
    stats_bytes = 4.0 * wl.R * wl.N * wl.D  # Q and K read once (bf16)

    # ---- back-to-back passes: each kernel family alone, every launch on another step's tensors (nothing is
    # L2-warm).  Inside a step the drift call follows the attention kernel, whose output is still being
    # written back from L2, and reads a few microseconds longer; both figures are reported.
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    st_b2b = heart.State(cfg, dev)
    st_b2b.load_state_dict(ckpt)
    torch.cuda.synchronize()
    a0.record()
    for k in range(K):
        Q, Kt, V = steps_in[W + k]
        heart.heart_drift(cfg, Q, Kt, delta, st_b2b, ws)
    a1.record()
    torch.cuda.synchronize()
    ms_drift_b2b = a0.elapsed_time(a1) / K
    del st_b2b
    f_last, _ = retained_flops(torch, st, wl)
    a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a0.record()
    for k in range(K):
        Q, Kt, V = steps_in[W + k]
        heart.heart_block_sparse_attn(cfg, Q, Kt, V, st.kv_idx, st.kv_cnt, O, ws)
    a1.record()
    torch.cuda.synchronize()
    ms_attn_b2b = a0.elapsed_time(a1) / K
    attn_tflops_b2b = float(f_last) / (ms_attn_b2b * 1e-3) / 1e12

    # ---- the same attention kernel with a full mask, measured where it fits in time (a dense run of the
    # two 720P shapes would take 0.1-0.15 s per launch): the sparse path's speedup over its own dense mode
    dense_ms = None
    if dense_flops < 3e13 and full:
        cfg_dense = heart.make_config(wl.B, wl.H, wl.N, wl.block, flags=heart.FORCE_DENSE)
        Q, Kt, V = steps_in[W]
        heart.heart_block_sparse_attn(cfg_dense, Q, Kt, V, None, None, O, ws)
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(3):
            heart.heart_block_sparse_attn(cfg_dense, Q, Kt, V, None, None, O, ws)
        b_.record()
        torch.cuda.synchronize()
        dense_ms = a.elapsed_time(b_) / 3

    # ---- mask prediction with every head refreshing, both estimators, on the first timed step's tensors:
    # the pooled one (the block means are in the workspace: heart_drift has just run) and the strided
    # antidiagonal one (a bf16 contraction per head on the tensor cores, in a workspace of its own size)
    Q, Kt, V = steps_in[W]
    st_m = heart.State(cfg, dev)

    def timed(fn, reps):
        fn()
        torch.cuda.synchronize()
        a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(reps):
            fn()
        b_.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b_) / reps

    heart.heart_drift(cfg, Q, Kt, delta, st_m, ws)
    ms_mask_pooled_all = timed(lambda: heart.heart_predict_mask(cfg, Q, Kt, tau, st_m, ws, means_valid=True), 5)
    dens_pooled = float(st_m.kv_cnt.to(torch.float64).mean()) / wl.n_blocks
    cfg_ad = heart.make_config(wl.B, wl.H, wl.N, wl.block, flags=heart.ESTIMATOR_ANTIDIAG)
    ws_ad = heart.new_workspace(cfg_ad, dev)
    ms_mask_ad_all = timed(lambda: heart.heart_predict_mask(cfg_ad, Q, Kt, tau, st_m, ws_ad), 3)
    assert heart.heart_get_status(ws_ad) == 0
    dens_ad = float(st_m.kv_cnt.to(torch.float64).mean()) / wl.n_blocks
    groups = wl.N // 16
    ad_flops = 2.0 * wl.R * float(groups) ** 2 * 16 * wl.D
    ad_ws_bytes = ws_ad.numel()
    del ws_ad, st_m

    hbm = stats_bytes / (ms_drift * 1e-3) / 1e9
    hbm_b2b = stats_bytes / (ms_drift_b2b * 1e-3) / 1e9
    l2_note = ("inputs larger than L2 (every step reads new Q/K/V tensors, >= 3x the 126 MB L2)"
               if 6 * wl.R * wl.N * wl.D > 126e6 else "L2-resident (tiny case): not a roofline number")
    region_ms = (ms_drift + ms_mask + ms_attn) * K
    rec = {
        "workload": wl.name, "config": config_of(wl), "steps": K, "warmup": W, "ms_per_step": ms_per_step,
        "l2": l2_note, "distinct_input_steps": n_inputs,
        "stages_ms": {"drift": ms_drift, "mask": ms_mask, "attention": ms_attn,
                      "sum_of_separate_calls": ms_drift + ms_mask + ms_attn},
        "mask_all_heads_ms": {"pooled": ms_mask_pooled_all, "strided_antidiagonal": ms_mask_ad_all,
                              "pooled_density": dens_pooled, "strided_antidiagonal_density": dens_ad,
                              "strided_antidiagonal_contraction_tflop": ad_flops / 1e12,
                              "strided_antidiagonal_tflops_whole_call": ad_flops / (ms_mask_ad_all * 1e-3) / 1e12,
                              "strided_antidiagonal_workspace_bytes": ad_ws_bytes},
        "density": density, "refresh_rate": refreshed / (K * wl.R),
        "retained_tflops": attn_tflops,
        "dense_equivalent_tflops": dense_flops / (ms_attn * 1e-3) / 1e12,
        "dense_equivalent_speedup_at_same_throughput": dense_flops / flops_step,
        "attention_ms_back_to_back": ms_attn_b2b, "retained_tflops_back_to_back": attn_tflops_b2b,
        "dense_attention_ms_measured": dense_ms,
        "dense_tflops_measured": (dense_flops / (dense_ms * 1e-3) / 1e12) if dense_ms else None,
        "attention_speedup_vs_measured_dense": (dense_ms / ms_attn) if dense_ms else None,
        "roofline": attention_roofline(pk, attn_tflops, clocks_stage, region_ms, flops_step, ms_attn,
                                       dram_traffic(wl.name)),
        "roofline_stats": {"kernel": "block sums + drift (heart_drift)", "bound": "hbm", "achieved": hbm,
                           "peak": pk["hbm_gbs"], "unit": "GB/s", "frac": hbm / pk["hbm_gbs"],
                           "frac_of_nominal_8TBps": hbm / 8000.0, "bytes_per_launch": stats_bytes,
                           "ms_per_launch": ms_drift, "peak_source": pk["source"] + " copy bandwidth",
                           "back_to_back": {"ms_per_launch": ms_drift_b2b, "achieved": hbm_b2b,
                                            "frac": hbm_b2b / pk["hbm_gbs"]}},
        "gpu_launches": launches, "wall_ms_timed_region": wall_ms, "clocks": clocks,
        "clocks_stage_pass": clocks_stage,
    }
    ctx = dict(wl=wl, steps_in=steps_in, W=W, K=K, cfg=cfg, st=st, ws=ws, ckpt=ckpt, delta=delta, tau=tau, O=O,
               barrier=barrier)
    return rec, ctx


def measure_e2e(torch, heart, replicas, ctx, dev, world):
    """Host (pinned) Q/K/V in, O/drift/refresh out, through heart_step_host."""
    wl, steps_in, W, K = ctx["wl"], ctx["steps_in"], ctx["W"], ctx["K"]
    cfg, st, ws, O = ctx["cfg"], ctx["st"], ctx["ws"], ctx["O"]
    Ke = min(K, max(1, int(6e9 // (4 * 2 * wl.R * wl.N * wl.D))))  # cap pinned memory at ~6 GB
    host_in = [tuple(x.cpu().pin_memory() for x in steps_in[W + k]) for k in range(Ke)]
    Oh = torch.empty(O.shape, dtype=O.dtype).pin_memory()
    dh = torch.empty(wl.R, dtype=torch.float64).pin_memory()
    rh = torch.empty(wl.R, dtype=torch.uint8).pin_memory()
    staging = tuple(torch.empty_like(O) for _ in range(4))
    st.load_state_dict(ctx["ckpt"])
    heart.heart_step_host(cfg, *host_in[0], ctx["delta"], ctx["tau"], st, Oh, staging, ws, drift_host=dh, refresh_host=rh)
    st.load_state_dict(ctx["ckpt"])
    ctx["barrier"]()
    a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for k in range(Ke):
        heart.heart_step_host(cfg, *host_in[k], ctx["delta"], ctx["tau"], st, Oh, staging, ws, drift_host=dh, refresh_host=rh)
    b_.record()
    ctx["barrier"]()
    e2e_ms = replicas.max_over_ranks(a.elapsed_time(b_) / Ke, dev)
    tensor_bytes = 2 * wl.R * wl.N * wl.D
    return {"value": replicas.job_ms_per_layer_step(e2e_ms, world), "unit": "ms", "steps": Ke,
            "h2d_bytes_per_step": 3 * tensor_bytes, "d2h_bytes_per_step": tensor_bytes + 9 * wl.R,
            "api": "heart_step_host (pinned host Q/K/V in, O + drift + refresh out)"}


def run_ours(args, rank, world):
    import gc

    import torch
    import torch.distributed as dist

    from paper_2605_14513_b200 import heart, inputs, replicas

    heart.lib()  # fails loudly if the CUDA library is missing
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    pk = peaks()
    wl = inputs.workload(args.workload)
    K, W = args.steps, args.warmup
    uuid = "GPU-" + str(torch.cuda.get_device_properties(dev).uuid).replace("GPU-", "")

    rec, ctx = measure(torch, heart, inputs, replicas, wl, K, W, dev, pk, rank, uuid, full=True)
    e2e = None if args.no_e2e else measure_e2e(torch, heart, replicas, ctx, dev, world)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(args, ctx["wl"], ctx["steps_in"], ctx["W"])
    del ctx
    gc.collect()
    torch.cuda.empty_cache()

    per = []
    if not args.no_per_workload and world == 1:
        names = [n for n in OTHERS + (HEADLINE,) if n != wl.name]
        for name in names:
            w2 = inputs.workload(name)
            k2 = min(K, 2 if w2.name == "tiny" else 6)
            r2, c2 = measure(torch, heart, inputs, replicas, w2, k2, 3, dev, pk, rank, uuid, full=False)
            del c2
            gc.collect()
            torch.cuda.empty_cache()
            per.append(r2)
        # the configuration text taken literally (positional scale 0.5): 83-98 % of the blocks are retained at
        # these thresholds, so the sparse path degenerates to near-dense attention; a secondary record
        lit = inputs.workload("wan1.3b-480p-literal")
        r2, c2 = measure(torch, heart, inputs, replicas, lit, min(K, 4), 3, dev, pk, rank, uuid, full=False)
        del c2
        gc.collect()
        torch.cuda.empty_cache()
        per.append(r2)

    out = None
    if rank == 0:
        out = {
            "metric": METRIC, "value": replicas.job_ms_per_layer_step(rec["ms_per_step"], world), "unit": "ms",
            "n_gpus": world, "steps": K, "warmup": W, "ms_per_step": rec["ms_per_step"], "higher_is_better": False,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": rec["config"], "parallelism": "replicas only" if world > 1 else "1 gpu", "l2": rec["l2"],
        }
        for k in ("stages_ms", "mask_all_heads_ms", "density", "refresh_rate", "retained_tflops", "dense_equivalent_tflops",
                  "dense_equivalent_speedup_at_same_throughput", "attention_ms_back_to_back",
                  "retained_tflops_back_to_back", "dense_attention_ms_measured", "dense_tflops_measured",
                  "attention_speedup_vs_measured_dense", "roofline", "roofline_stats", "gpu_launches",
                  "wall_ms_timed_region", "clocks", "clocks_stage_pass", "distinct_input_steps"):
            out[k] = rec[k]
        out["e2e"] = e2e
        if cpu is not None:
            out["cpu_baseline"] = cpu
        out["per_workload"] = [
            {"workload": r["workload"], "config": r["config"], "steps": r["steps"], "ms_per_step": r["ms_per_step"],
             "stages_ms": r["stages_ms"], "mask_all_heads_ms": r["mask_all_heads_ms"], "density": r["density"], "refresh_rate": r["refresh_rate"],
             "retained_tflops": r["retained_tflops"], "retained_tflops_back_to_back": r["retained_tflops_back_to_back"],
             "attention_frac": r["roofline"]["frac"], "attention_frac_of_burst_peak": r["roofline"]["frac_of_burst_peak"],
             "attention_frac_of_sustained_peak": r["roofline"]["frac_of_sustained_peak"],
             "attention_peak_used": r["roofline"]["peak_source"], "attention_dram_traffic": r["roofline"]["traffic"],
             "heart_drift_frac": r["roofline_stats"]["frac"],
             "heart_drift_frac_back_to_back": r["roofline_stats"]["back_to_back"]["frac"],
             "l2": r["l2"], "clocks": r["clocks"], "clocks_stage_pass": r["clocks_stage_pass"]} for r in per]
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()
    return out


def sample_rows_for(wl, requested):
    """Query blocks the oracle attends per step: about a second of CPU work on ~16 cores."""
    if requested > 0:
        return requested
    keys_per_row = 0.12 * wl.n_blocks * wl.block  # ~12 % density
    flop_per_row = 4.0 * wl.block * keys_per_row * wl.D
    return int(max(8, min(384, 3.0e10 // flop_per_row)))


def oracle_sample_step(oracle, np, wl, ost, Qb, Kb, Vb, rs, n_rows):
    """One oracle layer-step on a bounded sample: drift + decision + masks in full, attention on
    n_rows query blocks, its time scaled by retained pairs.  Returns (seconds extrapolated, seconds spent)."""
    t0 = time.perf_counter()
    oracle.step(Qb, Kb, Vb, wl.delta, wl.tau, ost, want_O=False)
    t1 = time.perf_counter()
    rr = rs.randint(0, wl.R, n_rows).astype(np.int32)
    II = rs.randint(0, wl.n_blocks, n_rows).astype(np.int32)
    oracle.attn_rows(Qb, Kb, Vb, wl.block, ost.kv_idx, ost.kv_cnt, rr, II)
    t2 = time.perf_counter()
    sampled = float(ost.kv_cnt[rr, II].sum())
    scale = float(ost.kv_cnt.sum()) / max(sampled, 1.0)
    return (t1 - t0) + (t2 - t1) * scale, t2 - t0


def run_reference(args):
    """The oracle as it stands, on the host cores (rank 0 only).  The synthetic inputs are generated
    on the GPU when there is one (the generator is shared by both arms and is not timed), else on the
    CPU; everything timed is the oracle on the host."""
    import numpy as np
    import torch

    from oracle import heart_oracle as oracle
    from paper_2605_14513_b200 import inputs

    oracle.build()
    wl = inputs.workload(args.workload)
    K, W = args.steps, args.warmup
    gen_dev = "cuda" if torch.cuda.is_available() else "cpu"
    seq = inputs.Sequence(wl, gen_dev)
    ost = oracle.State(wl.B, wl.H, wl.N, wl.D, wl.block)
    rs = np.random.RandomState(0)
    n_rows = sample_rows_for(wl, args.cpu_sample_rows)
    est, spent = [], 0.0
    for t in range(W + K):
        Qb, Kb, Vb = (inputs.bits(x) for x in seq.bf16())
        e, s = oracle_sample_step(oracle, np, wl, ost, Qb, Kb, Vb, rs, n_rows)
        if t >= W:
            est.append(e)
            spent += s
        if t + 1 < W + K:
            seq.advance()
    ms = 1e3 * sum(est) / K
    cores = os.cpu_count()
    sample = (f"per step: token means, decision and masks in full; attention on {n_rows} random "
              f"query blocks scaled by retained pairs ({spent:.1f} s of CPU work in {K} steps)")
    return {"impl": "reference", "metric": METRIC, "value": ms, "unit": "ms", "n_gpus": args.gpus, "steps": K,
            "warmup": W, "ms_per_step": ms, "higher_is_better": False, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64", "data": "synthetic", "config": config_of(wl), "extrapolated": True,
            "cpu_seconds_spent_in_timed_steps": spent,
            "cpu_baseline": {"value": ms, "unit": "ms", "cores": cores, "kind": "oracle", "sample": sample,
                             "extrapolated": True},
            "e2e": {"value": ms, "unit": "ms", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}


def cpu_baseline(args, wl, steps_in, W):
    """The oracle timed on the host cores on a bounded sample of the benchmark's own inputs."""
    import numpy as np

    from oracle import heart_oracle as oracle
    from paper_2605_14513_b200 import inputs

    oracle.build()
    ost = oracle.State(wl.B, wl.H, wl.N, wl.D, wl.block)
    rs = np.random.RandomState(0)
    n_rows = sample_rows_for(wl, args.cpu_sample_rows)
    est, spent, n = [], 0.0, 0
    budget = 20.0
    # step 0 builds the anchors and masks (all heads refresh); later steps show the steady mix
    for t in range(min(len(steps_in), W + 3)):  # (a cycled input pool repeats only beyond W + 3 steps here)
        Qb, Kb, Vb = (inputs.bits(x) for x in steps_in[t])
        e, s = oracle_sample_step(oracle, np, wl, ost, Qb, Kb, Vb, rs, n_rows)
        spent += s
        if t >= 1:
            est.append(e)
        n += 1
        if spent > budget:
            break
    if not est:
        est = [e]
    ms = 1e3 * sum(est) / len(est)
    return {"value": ms, "unit": "ms", "cores": os.cpu_count(), "kind": "oracle", "extrapolated": True,
            "sample": (f"{n} steps of the same inputs ({len(est)} after the all-refresh first step averaged); per step: "
                       f"token means, decision and masks in full, attention on {n_rows} random query blocks "
                       f"scaled by retained pairs; {spent:.1f} s of CPU work")}


def spawn_ranks(n):
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one process per GPU)."""
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    args = parse()
    rank = int(os.environ.get("RANK", 0))
    if args.impl == "reference":
        if rank == 0:
            print(json.dumps(run_reference(args)), flush=True)
        return 0
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        return spawn_ranks(args.gpus)
    world = int(os.environ.get("WORLD_SIZE", 1))
    if world != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world}: launch one rank per GPU", file=sys.stderr)
        return 2
    out = run_ours(args, rank, world)
    if rank == 0:
        print(json.dumps(out), flush=True)
    return 0


if __name__ == "__main__":
    sys.exit(main())

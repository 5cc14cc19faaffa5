#!/usr/bin/env python
"""Benchmark of gc_build_cache (Step 2 of Gradient Cache: loss + representation gradients).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--config I]

One "step" is one gc_build_cache call over one synthetic batch.  The default workload is the
headline configuration B = 4096, N = 8192, d = 768, bf16 inputs.  The metric is useful TFLOP/s
counting 3 GEMMs of 2 B N d each.  With N > 1 the ONE batch is split over the ranks the way
Section 3.4 of the paper describes (all-gather of the representations, rank-local gradients,
exchange of the row logsumexps): strong scaling, collectives inside the timed region.
`--parallel replicas` runs N independent batches instead (weak scaling, no collective).
`--gpus N` without a torchrun environment starts the N ranks itself.

Prints ONE JSON line on rank 0.  `--impl reference` times the CPU oracle instead (a deliberately
plain program; see oracle/).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

UNIT = "TFLOP/s"


def metric_name(B, N, d):
    return f"gc_build_cache TFLOP/s (3 GEMMs of 2*B*N*d) at B={B},N={N},d={d}"


NOMINAL_BF16_TFLOPS = 2250.0      # public dense bf16 figure for B200, context only
# dram__bytes_read.sum + dram__bytes_write.sum of ONE STEP (every launch of a gc_build_cache
# call summed) from the ncu captures summarised under profiles/ (quad_kernel_cfg2_*, quad_kernel_
# cfg4_*, small_kernel_*).  Under ncu every launch starts from flushed caches, so a step of
# several launches counts its inputs once per launch.  A figure is reported only while the
# sources its kernels come from still have the hash they had when the counters were taken.
SWEEP_SOURCES = ['gc_api.cu', 'gc_combine.cu', 'gc_internal.h', 'gc_quad.cu', 'gc_tc.cu', 'tc_common.cuh']
ONE_TILE_SOURCES = ['gc_api.cu', 'gc_internal.h', 'gc_small.cu', 'tc_common.cuh']
NARROW_SOURCES = SWEEP_SOURCES + ['gc_narrow.cu']
NCU_STEP_TRAFFIC = {
    "cfg2_": (82.9e6, SWEEP_SOURCES, "984da4d026488e42db1a380f3e3a5b542047d09f"),
    "cfg4_": (4.80e9, SWEEP_SOURCES, "984da4d026488e42db1a380f3e3a5b542047d09f"),
    "cfg3_": (26.4e6, NARROW_SOURCES, "44a0d1324795e9d77b5ed87232933502e92ce031"),
    "cfg1_": (0.629e6, ONE_TILE_SOURCES, "42794198880e3035735ceb1c20a53113fbce4c0e"),
    "cfg0_": (0.640e6, ONE_TILE_SOURCES, "42794198880e3035735ceb1c20a53113fbce4c0e"),
}
FP32_LANES_PER_SM = 128           # fp32 FMA lanes of one SM (2 FLOP per lane and clock)


def sources_sha1(files):
    import hashlib
    h = hashlib.sha1()
    for f in files:
        with open(os.path.join(ROOT, "paper_2101_06983_b200", "csrc", f), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()


def ncu_traffic(workload: str):
    for prefix, (val, files, digest) in NCU_STEP_TRAFFIC.items():
        if workload.startswith(prefix):
            try:
                return val if sources_sha1(files) == digest else None
            except OSError:
                return None
    return None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            pk = json.load(fh)
        return dict(hbm=float(pk["hbm_gbs"]), tf_burst=float(pk["bf16_tflops"]),
                    tf_sustained=float(pk.get("bf16_tflops_sustained", pk["bf16_tflops"])),
                    source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


def useful_flop(B, N, d):
    return 3.0 * 2.0 * B * N * d


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs
    (read-only queries)."""

    def __init__(self, index: int, period: float = 0.002):
        super().__init__(daemon=True)
        self.index, self.period = index, period
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self.stop_flag = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:          # NVML missing: report nulls
            self.ok = False

    def sample_once(self):
        """One synchronous sample (called from the timed loop while a step is executing)."""
        if not self.ok:
            return
        nv = self.nv
        try:
            self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
            mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
            for name in ("HwSlowdown", "HwThermalSlowdown", "SwThermalSlowdown", "SwPowerCap"):
                if mask & getattr(nv, "nvmlClocksThrottleReason" + name):
                    self.reasons.add({"HwSlowdown": "hw_slowdown",
                                      "HwThermalSlowdown": "hw_thermal_slowdown",
                                      "SwThermalSlowdown": "sw_thermal_slowdown",
                                      "SwPowerCap": "sw_power_cap"}[name])
        except Exception:
            pass

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
            nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
            nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap",
            nv.nvmlClocksThrottleReasonHwPowerBrakeSlowdown: "hw_power_brake",
        }
        while not self.stop_flag.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def result(self):
        self.stop_flag.set()
        if self.is_alive():
            self.join(timeout=2.0)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": []}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def physical_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except (ValueError, IndexError):
            return local_rank
    return local_rank


def run_reference(args, rank, world):
    """CPU oracle timed as it stands on a bounded sample of the workload."""
    if rank != 0:
        return
    import oracle
    from paper_2101_06983_b200 import inputs
    prob = inputs.config(args.config)
    rows = max(1, min(prob.B, args.ref_rows, int(2.6e10 / (prob.N * prob.d))))
    Q, pos = prob.Q[:rows], prob.pos_idx[:rows]
    flop = useful_flop(rows, prob.N, prob.d)
    for _ in range(args.warmup):
        oracle.build_cache(Q, prob.P, pos, prob.tau, prob.mask_mode)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle.build_cache(Q, prob.P, pos, prob.tau, prob.mask_mode)
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = flop / dt / 1e12
    sample = (f"first {rows} of {prob.B} query rows against all {prob.N} passages "
              f"(loss, dQ rows, dP contributions), double precision, per step")
    line = {
        "impl": "reference", "metric": metric_name(prob.B, prob.N, prob.d), "value": value,
        "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": prob.name, "B": prob.B, "N": prob.N, "d": prob.d,
                   "sample_rows": rows},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, rank, local_rank, world):
    import torch
    import torch.distributed as dist

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    from paper_2101_06983_b200 import binding, replicas

    prob = replicas.replica_problem(args.config, rank)
    B, N, d = prob.B, prob.N, prob.d
    code = binding.GC_BF16 if prob.dtype == "bf16" else binding.GC_F32
    Q, P, pos = binding.problem_tensors(prob, dev)
    stored = args.plan == "stored"
    op = binding.GC_OP_BUILD_STORED if stored else binding.GC_OP_BUILD
    build = binding.gc_build_cache_stored if stored else binding.gc_build_cache
    out = binding.Outputs(B, N, d, code, dev, op)
    flop = useful_flop(B, N, d)
    plan = binding.gc_plan_name(binding.GC_OP_BUILD, B, N, d, code) + ("+stored" if stored else "")
    launches = binding.gc_kernel_launches(op, B, N, d, code)

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)   # larger than the 126 MB L2

    def step():
        build(Q, P, pos, prob.tau, prob.mask_mode, out.loss, out.row_lse, out.dQ, out.dP,
              out.pos_logit, out.ws, out.dev_status)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: every step starts with a cold L2 ---------------------------
    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        step()
    barrier()
    # All timed steps are queued without a host synchronisation in between.  Two passes of the
    # same K flushed steps: the first, without per-kernel events, gives the step time; the second
    # has the library bracket its sweep kernels with CUDA events on the launching stream (one
    # event set per call) and gives their durations.  The events cost a step about 15 us (each
    # one drains the stream, and the one between the anchor kernel and the fused sweep keeps the
    # sweep from starting early), which is why the step time is not taken from that pass.
    def timed_pass(with_kernel_events: bool):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(args.steps)]
        kern = [0.0, 0.0, 0.0]
        done = 0
        while done < args.steps:
            chunk = min(256, args.steps - done)
            if with_kernel_events:
                binding.gc_profile_enable(chunk)
            for a, b in ev[done:done + chunk]:
                flush.fill_(1)
                a.record()
                step()
                b.record()
            torch.cuda.synchronize()
            if with_kernel_events:
                for c in range(chunk):
                    ms = binding.gc_profile_read(c)
                    for k in range(3):
                        kern[k] += ms[k]
            done += chunk
        binding.gc_profile_enable(False)
        return sum(a.elapsed_time(b) for a, b in ev), kern

    sampler = ClockSampler(physical_gpu_index(local_rank), period=0.0005)
    sampler.start()
    total_ms, _ = timed_pass(False)
    barrier()
    profiled_ms, kern = timed_pass(True)
    barrier()
    clocks = sampler.result()

    # ---- back-to-back timing (inputs and outputs stay in L2, as right after an encoder) -------
    barrier()
    a = torch.cuda.Event(enable_timing=True)
    b = torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(args.steps):
        step()
    b.record()
    barrier()
    warm_ms = a.elapsed_time(b) / args.steps

    # ---- the same step replayed from a CUDA graph (captured once: the call is capturable, its
    # side-stream work is forked from and joined back into the capturing stream) ----------------
    graph_block = None
    if not args.no_graph:
        try:
            gs = torch.cuda.Stream()
            gs.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(gs):
                step()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=gs):
                step()
            for _ in range(3):
                flush.fill_(1)
                g.replay()
            ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                  for _ in range(args.steps)]
            for ea, eb in ev:
                flush.fill_(1)
                ea.record()
                g.replay()
                eb.record()
            torch.cuda.synchronize()
            g_ms = sum(ea.elapsed_time(eb) for ea, eb in ev) / args.steps
            ea = torch.cuda.Event(enable_timing=True)
            eb = torch.cuda.Event(enable_timing=True)
            ea.record()
            for _ in range(args.steps):
                g.replay()
            eb.record()
            torch.cuda.synchronize()
            g_warm = ea.elapsed_time(eb) / args.steps
            graph_block = {"ms_per_step": g_ms, "value": flop / (g_ms * 1e-3) / 1e12, "unit": UNIT,
                           "warm_l2_ms_per_step": g_warm,
                           "note": "one gc_build_cache call captured into a CUDA graph and replayed; "
                                   "L2 flushed before every timed replay"}
            del g
        except RuntimeError as exc:            # capture refused: report it, keep the eager numbers
            graph_block = {"error": str(exc)[:200]}
        barrier()

    # ---- sustained: at least a second of back-to-back steps, clocks sampled meanwhile -------------
    # A short timed region runs at boost clocks; under a second of tensor work the power cap
    # settles the SM clock lower.  time x median MHz lets runs at different clocks be compared.
    sustained = None
    if not args.no_sustained:
        n_sus = max(args.steps, int(1.2 / max(warm_ms * 1e-3, 1e-6)))
        sus_sampler = ClockSampler(physical_gpu_index(local_rank), period=0.005)
        barrier()
        sus_sampler.start()
        a.record()
        for _ in range(n_sus):
            step()
        b.record()
        barrier()
        sus_clocks = sus_sampler.result()
        sus_ms = a.elapsed_time(b) / n_sus
        sustained = {"steps": n_sus, "ms_per_step": sus_ms,
                     "value": world * flop / (sus_ms * 1e-3) / 1e12, "unit": UNIT,
                     "sm_mhz_median": sus_clocks["sm_mhz"], "reasons": sus_clocks["reasons"],
                     "ms_x_mhz": None if sus_clocks["sm_mhz"] is None
                     else sus_ms * sus_clocks["sm_mhz"]}

    # ---- end to end through the C ABI with host buffers ------------------------------------------
    # Every step copies its inputs from pinned host memory, calls gc_build_cache and copies the
    # cache (dQ, dP) and the loss back.  Two sets of device buffers and three streams (upload,
    # compute, download) let the copies of neighbouring steps overlap the kernels; each step's
    # own upload -> compute -> download order is kept by events.
    hQ = Q.cpu().pin_memory()
    hP = hQ if prob.shared else P.cpu().pin_memory()
    hpos = pos.cpu().pin_memory()
    NB = 2
    h_out = [(torch.empty(out.dQ.shape, dtype=torch.float32).pin_memory(),
              torch.empty(out.dP.shape, dtype=torch.float32).pin_memory(),
              torch.empty(1, dtype=torch.float32).pin_memory()) for _ in range(NB)]
    d_in = []
    for _ in range(NB):
        q_ = torch.empty_like(Q)
        d_in.append((q_, q_ if prob.shared else torch.empty_like(P), torch.empty_like(pos)))
    d_out = [out] + [binding.Outputs(B, N, d, code, dev, op) for _ in range(NB - 1)]
    s_up, s_run, s_down = (torch.cuda.Stream(dev) for _ in range(3))
    ev_up = [torch.cuda.Event() for _ in range(NB)]
    ev_run = [torch.cuda.Event() for _ in range(NB)]
    ev_down = [torch.cuda.Event() for _ in range(NB)]

    def e2e_step(i):
        k = i % NB
        with torch.cuda.stream(s_up):
            s_up.wait_event(ev_run[k])            # the previous user of these inputs has run
            d_in[k][0].copy_(hQ, non_blocking=True)
            if not prob.shared:
                d_in[k][1].copy_(hP, non_blocking=True)
            d_in[k][2].copy_(hpos, non_blocking=True)
            ev_up[k].record(s_up)
        with torch.cuda.stream(s_run):
            s_run.wait_event(ev_up[k])
            s_run.wait_event(ev_down[k])          # the previous results of this set are out
            o = d_out[k]
            build(d_in[k][0], d_in[k][1], d_in[k][2], prob.tau, prob.mask_mode, o.loss, o.row_lse,
                  o.dQ, o.dP, o.pos_logit, o.ws, o.dev_status)
            ev_run[k].record(s_run)
        with torch.cuda.stream(s_down):
            s_down.wait_event(ev_run[k])
            h_out[k][0].copy_(d_out[k].dQ, non_blocking=True)
            h_out[k][1].copy_(d_out[k].dP, non_blocking=True)
            h_out[k][2].copy_(d_out[k].loss, non_blocking=True)
            ev_down[k].record(s_down)

    e2e_steps = max(4, min(args.steps, 20))
    for i in range(2 * NB):
        e2e_step(i)
    barrier()
    a.record()
    for i in range(e2e_steps):
        e2e_step(i)
    for st_ in (s_up, s_run, s_down):
        torch.cuda.current_stream().wait_stream(st_)
    b.record()
    barrier()
    e2e_ms = a.elapsed_time(b) / e2e_steps
    e2e_loss = float(h_out[(e2e_steps - 1) % NB][2].item())
    h2d = hQ.numel() * hQ.element_size() + (0 if prob.shared else hP.numel() * hP.element_size()) \
        + hpos.numel() * 4
    d2h = (h_out[0][0].numel() + h_out[0][1].numel() + 1) * 4
    status = int(out.dev_status.item())

    # ---- max over ranks ------------------------------------------------------------------------------
    total_ms, warm_ms, e2e_ms = replicas.max_over_ranks([total_ms, warm_ms, e2e_ms], dev)
    ms_per_step = total_ms / args.steps

    if rank == 0:
        pk = load_peaks()
        # dominant kernel: the tile sweep kernel, launched twice per step for the gradients.  The
        # dP launch delivers one useful GEMM (2 B N d); the dQ launch delivers one, or two when the
        # forward is fused into it (no separate forward launch was timed).
        # The stored-weights plan has three tensor kernels of one useful GEMM each.
        fused = kern[0] == 0.0
        if stored:
            sweep_ms = (kern[0] + kern[1] + kern[2]) / (3 * args.steps)
            sweep_flop = 2.0 * B * N * d
        else:
            sweep_ms = (kern[1] + kern[2]) / (2 * args.steps)
            sweep_flop = (6.0 if fused else 4.0) * B * N * d / 2.0      # per launch, averaged
        achieved = sweep_flop / (sweep_ms * 1e-3) / 1e12 if sweep_ms > 0 else 0.0
        value = replicas.whole_job_rate(flop, world, ms_per_step) / 1e12
        if plan.startswith("tcgen05"):
            roof = {"bound": "tensor", "kernel": f"{plan} sweeps (the tensor-core launches of a step)",
                    "achieved": achieved, "peak": pk["tf_burst"], "unit": "TFLOP/s",
                    "frac": achieved / pk["tf_burst"], "peak_source": pk["source"]}
        else:
            # fp32 FMA tiles: bound by the fp32 pipes, SMs x 128 lanes x 2 FLOP x the maximum SM
            # clock; the launches of a step executed (fwd 2 + dQ 4 + dP 4) B N d
            alu_ms = (kern[0] + kern[1] + kern[2]) / args.steps
            executed = 10.0 * B * N * d / (alu_ms * 1e-3) / 1e12 if alu_ms > 0 else 0.0
            sms = torch.cuda.get_device_properties(dev).multi_processor_count
            mhz = clocks["sm_max_mhz"] or 1965
            alu_peak = sms * FP32_LANES_PER_SM * 2 * mhz * 1e6 / 1e12
            roof = {"bound": "alu", "kernel": "fp32 FMA tile kernels (forward, dQ and dP sweeps)",
                    "achieved": executed, "peak": alu_peak, "unit": "TFLOP/s",
                    "frac": executed / alu_peak,
                    "peak_source": "derived: SMs x 128 fp32 lanes x 2 x max SM clock"}
        step_traffic = None if stored else ncu_traffic(prob.name)
        roof["traffic"] = step_traffic
        roof["traffic_scope"] = "dram bytes of one step, all launches (ncu)"
        roof["algorithmic_bytes_per_step"] = (B + N) * d * (2 if prob.dtype == "bf16" else 4) + \
            (B + N) * d * 4
        line = {
            "metric": metric_name(B, N, d), "value": value, "unit": UNIT, "n_gpus": world,
            "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if prob.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": prob.name, "B": B, "N": N, "d": d, "tau": prob.tau,
                       "mask": "self" if prob.mask_mode else "none", "plan": plan,
                       "l2": "flushed before every timed step (256 MiB write)",
                       "parallelism": f"{world} independent replica(s), no collective"},
            "rows_per_s": world * (B + N) / (ms_per_step * 1e-3),
            "pct_of_bf16_peak": {"burst_measured": 100 * value / world / pk["tf_burst"],
                                 "sustained_measured": 100 * value / world / pk["tf_sustained"],
                                 "nominal_dense": 100 * value / world / NOMINAL_BF16_TFLOPS,
                                 "peaks": pk["source"]},
            "graph": graph_block,
            "warm_l2": {"ms_per_step": warm_ms,
                        "value": world * flop / (warm_ms * 1e-3) / 1e12, "unit": UNIT},
            "kernel_ms": {"fwd_sweep": kern[0] / args.steps, "dq_sweep": kern[1] / args.steps,
                          "dp_sweep": kern[2] / args.steps,
                          "pass": "second pass of the same flushed steps, per-kernel CUDA events",
                          "ms_per_step_with_events": profiled_ms / args.steps},
            "sustained": sustained,
            "roofline": roof,
            "e2e": {"value": world * flop / (e2e_ms * 1e-3) / 1e12, "unit": UNIT,
                    "ms_per_step": e2e_ms, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "loss_read_back": e2e_loss,
                    "pipeline": "2 buffer sets; upload, compute and download streams"},
            "gpu_launches": launches * args.steps,
            "clocks": clocks, "dev_status": status, "loss": float(out.loss.item()),
        }
        if world == 1 and not args.no_cpu_baseline:
            import oracle
            rows = max(1, min(B, args.ref_rows, int(2.6e10 / (N * d))))   # about 10-30 s
            t0 = time.perf_counter()
            ref = oracle.build_cache(prob.Q[:rows], prob.P, prob.pos_idx[:rows], prob.tau,
                                     prob.mask_mode)
            dt = time.perf_counter() - t0
            line["cpu_baseline"] = {
                "value": useful_flop(rows, N, d) / dt / 1e12, "unit": UNIT,
                "cores": oracle.num_threads(), "kind": "oracle", "seconds": dt,
                "sample": f"first {rows} of {B} query rows against all {N} passages, one pass, "
                          f"double precision"}
            if rows == B:
                line["loss_rel_err_vs_oracle"] = abs(line["loss"] - ref["loss"]) / abs(ref["loss"])
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_sharded(args, rank, local_rank, world):
    """Multi-GPU mode (default for N > 1): ONE global batch of the chosen workload is split over
    the ranks as Section 3.4 describes (all-gather of representations, rank-local forward + dQ
    and dP, exchange of row_lse, loss all-reduce).  Strong scaling: the value is the whole batch's
    useful FLOP over the slowest rank's time, collectives included."""
    import torch
    import torch.distributed as dist
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
    from paper_2101_06983_b200 import binding, inputs, replicas, sharded

    def measure(index, steps, warmup):
        prob = inputs.config(index)
        B, N, d = prob.B, prob.N, prob.d
        Q, P, pos = binding.problem_tensors(prob, dev)
        (q0, b), (p0, n) = sharded.row_ranges(B, world)[rank], sharded.row_ranges(N, world)[rank]
        Ql, Pl = Q[q0:q0 + b].contiguous(), P[p0:p0 + n].contiguous()
        posl = pos[q0:q0 + b].contiguous()
        del Q, P, pos
        step = sharded.ShardedStep(B, N, d, Ql.dtype, dev, mask_mode=prob.mask_mode)

        def barrier():
            if world > 1:
                dist.barrier()
            torch.cuda.synchronize()

        for _ in range(max(warmup, 3)):
            step.run(Ql, Pl, posl, prob.tau)
        barrier()
        a, bev = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(steps):
            loss = step.run(Ql, Pl, posl, prob.tau)[0]
        bev.record()
        barrier()
        ms = replicas.max_over_ranks([a.elapsed_time(bev) / steps], dev)[0]
        # where the time goes: one more pass with every section synchronised (diagnostic)
        parts = {"gather_reps_s": 0.0, "fwd_dq_s": 0.0, "lse_and_loss_s": 0.0, "dp_s": 0.0}
        for _ in range(3):
            step.run(Ql, Pl, posl, prob.tau, measure=True)
            for k in parts:
                parts[k] += step.timings[k] / 3
        keys = sorted(parts)
        worst = replicas.max_over_ranks([parts[k] for k in keys], dev)
        comm = sum(v for k, v in zip(keys, worst) if k in ("gather_reps_s", "lse_and_loss_s"))
        comp = sum(v for k, v in zip(keys, worst) if k in ("fwd_dq_s", "dp_s"))
        return prob, ms, float(loss.item()), {"communication_ms": comm * 1e3,
                                              "compute_ms": comp * 1e3,
                                              "note": "sections synchronised one by one, max over ranks"}

    prob, ms, loss, split = measure(args.config, args.steps, args.warmup)
    also = None
    if world > 1 and args.config != 4 and not args.no_also:
        p4, ms4, loss4, split4 = measure(4, max(3, min(args.steps, 5)), 3)
        also = {"workload": p4.name, "ms_per_step": ms4,
                "value": useful_flop(p4.B, p4.N, p4.d) / (ms4 * 1e-3) / 1e12, "unit": UNIT,
                "loss": loss4, "split": split4}
    if rank == 0:
        B, N, d = prob.B, prob.N, prob.d
        flop = useful_flop(B, N, d)
        print(json.dumps({
            "metric": metric_name(B, N, d), "value": flop / (ms * 1e-3) / 1e12, "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
            "higher_is_better": True, "scaling": "strong", "vs_baseline": None,
            "dtype": "bf16" if prob.dtype == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": prob.name, "B": B, "N": N, "d": d,
                       "parallelism": f"query and passage rows sharded over {world} rank(s), "
                                      "Section 3.4: all-gather of Q, P, pos_idx; all-gather of "
                                      "row_lse; all-reduce of the loss",
                       "l2": "back to back, no flush (collectives between the kernels)"},
            "split": split, "also": also, "loss": loss,
            "gpu_launches": args.steps * (
                binding.gc_kernel_launches(binding.GC_OP_BUILD, max(1, B // world), N, d,
                                           binding.GC_BF16 if prob.dtype == "bf16" else binding.GC_F32)
                + 3)}), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_apply(args):
    """Side measurement (not the headline metric): gc_cache_apply, Step 3 for a linear encoder,
    dW (+)= U^T X over one sub-batch of --apply-rows rows with d = d_in = 768.  HBM-bound by its
    algorithmic bytes (U fp32 and X bf16 read once, dW fp32 written once)."""
    import numpy as np
    import torch
    from paper_2101_06983_b200 import binding, inputs
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the library has no CPU path")
    rows, d, d_in = args.apply_rows, 768, 768
    U = inputs.cache_rows(rows, d, seed=1)
    xbits, X = inputs.encoder_inputs(rows, d_in, seed=2)
    dU = torch.from_numpy(U).cuda()
    dX = torch.from_numpy(xbits.view(np.int16)).view(torch.bfloat16).cuda()
    dW = torch.empty(d, d_in, device="cuda")
    ws = torch.empty(binding.gc_cache_apply_workspace_bytes(rows, d, d_in), dtype=torch.uint8,
                     device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    for _ in range(max(args.warmup, 3)):
        flush.fill_(1)
        binding.gc_cache_apply(dU, dX, dW, False, ws)
    torch.cuda.synchronize()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
          for _ in range(args.steps)]
    for a, b in ev:
        flush.fill_(1)
        a.record()
        binding.gc_cache_apply(dU, dX, dW, False, ws)
        b.record()
    torch.cuda.synchronize()
    ms = sum(a.elapsed_time(b) for a, b in ev) / args.steps
    pk = load_peaks()
    nbytes = 4.0 * rows * d + 2.0 * rows * d_in + 4.0 * d * d_in
    # dram bytes of the call's one launch at 4096 rows, from
    # profiles/apply_kernel_rows4096_d768_din768.txt; reported while gc_apply.cu is unchanged
    import hashlib
    with open(os.path.join(ROOT, "paper_2101_06983_b200", "csrc", "gc_apply.cu"), "rb") as fh:
        same = hashlib.sha1(fh.read()).hexdigest() == "71def43a9090e7af98d500aed9dc7b0ff9170948"
    traffic = 18.9e6 if same and rows == 4096 else None
    import oracle
    t0 = time.perf_counter()
    ref = oracle.cache_apply(U, X)
    dt = time.perf_counter() - t0
    err = float(np.abs(dW.cpu().numpy() - ref).max() / np.abs(ref).max())
    line = {
        "metric": f"gc_cache_apply rows/s at rows={rows},d={d},d_in={d_in}", "value": rows / (ms * 1e-3),
        "unit": "rows/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms, "higher_is_better": True, "dtype": "bf16 x (bf16 + bf16), fp32 accumulate",
        "data": "synthetic",
        "config": {"workload": f"apply_rows{rows}_d{d}_din{d_in}",
                   "l2": "flushed before every timed step (256 MiB write)"},
        "tflops": 2.0 * rows * d * d_in / (ms * 1e-3) / 1e12,
        "roofline": {"bound": "hbm", "achieved": nbytes / (ms * 1e-3) / 1e9, "peak": pk["hbm"],
                     "unit": "GB/s", "frac": nbytes / (ms * 1e-3) / 1e9 / pk["hbm"],
                     "peak_source": pk["source"], "traffic": traffic},
        "cpu_baseline": {"value": rows / dt, "unit": "rows/s", "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": "the same sub-batch, one pass, double precision"},
        "max_err_vs_oracle": err, "gpu_launches": args.steps,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", type=int, default=2, help="workload index 0..4 (2 = headline)")
    ap.add_argument("--ref-rows", type=int, default=None,
                    help="query rows in the CPU sample (default: whole batch for ours' "
                         "cpu_baseline, 512 for --impl reference)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--plan", default="recompute", choices=["recompute", "stored"],
                    help="recompute: gc_build_cache (nothing of size B x N leaves the chip); "
                         "stored: gc_build_cache_stored, the comparison plan that keeps the "
                         "B x N bf16 weights in the workspace")
    ap.add_argument("--op", default="build", choices=["build", "apply"],
                    help="build: gc_build_cache, the headline; apply: the side measurement of "
                         "gc_cache_apply (one GPU)")
    ap.add_argument("--apply-rows", type=int, default=4096)
    ap.add_argument("--parallel", default=None, choices=["replicas", "shard"],
                    help="shard (default for N > 1): one batch split over the ranks as in Section "
                         "3.4 of the paper, strong scaling; replicas (default for N = 1): "
                         "independent batches, weak scaling, no collective")
    ap.add_argument("--no-graph", action="store_true",
                    help="skip the CUDA-graph replay of the step")
    ap.add_argument("--no-sustained", action="store_true",
                    help="skip the second-long back-to-back measurement")
    ap.add_argument("--no-also", action="store_true",
                    help="sharded mode: skip the B=65536 workload measured beside the chosen one")
    args = ap.parse_args()
    env_world = os.environ.get("WORLD_SIZE")
    if env_world is not None and int(env_world) != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} contradicts WORLD_SIZE={env_world}")
    if args.gpus > 1 and env_world is None and args.impl == "ours" and args.op == "build":
        # not under torchrun: start the ranks ourselves, one per GPU of this node
        import torch
        have = torch.cuda.device_count() if torch.cuda.is_available() else 0
        if have < args.gpus:
            raise SystemExit(f"--gpus {args.gpus} needs {args.gpus} CUDA devices on this node, "
                             f"found {have}: refusing to run fewer ranks")
        import socket
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
        os.execv(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                                  f"--nproc-per-node={args.gpus}", "--master-addr", "127.0.0.1",
                                  "--master-port", str(port), os.path.abspath(__file__),
                                  *sys.argv[1:]])
    if args.parallel is None:
        args.parallel = "shard" if args.gpus > 1 else "replicas"
    if args.op == "apply":
        if int(os.environ.get("RANK", "0")) == 0:
            run_apply(args)
        return
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        if args.ref_rows is None:
            args.ref_rows = 512
        run_reference(args, rank, world)
        return
    if args.ref_rows is None:
        args.ref_rows = 4096
    if args.parallel == "shard":
        run_sharded(args, rank, local_rank, world)
        return
    run_ours(args, rank, local_rank, world)


if __name__ == "__main__":
    main()

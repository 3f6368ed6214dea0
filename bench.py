#!/usr/bin/env python
"""Benchmark of the MoE layer hot path: one step = moe_forward + moe_backward (both balancing
losses included) over one synthetic batch.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config c5] [--impl ours|reference]

N > 1 is launched by torchrun (one rank per GPU); the layer has no exchange step on one GPU per
replica, so ranks run independent replicas ("weak" scaling, no data-path collective); timing is the
max over ranks. Prints ONE JSON line on rank 0.
"""
from __future__ import annotations

import argparse
import concurrent.futures
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_1701_06538_b200 import replicas, synth  # noqa: E402

METRIC = "moe_layer_fwd_bwd_tokens_per_s"
UNIT = "tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
L2_BYTES = 126 * 2 ** 20
# FP32 FMA peak of a B200 at its maximum SM clock: 148 SMs x 128 lanes x 2 flop x 1.965 GHz
FP32_PEAK_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12
# dram__bytes_read.sum + dram__bytes_write.sum of the six expert GEMMs of one step come from an ncu capture whose summary
# under profiles/ records the figure per workload together with the hash of the GEMM source it was taken with: a figure
# taken with another version of the kernels is not reported (null) rather than carried along
TRAFFIC_SUMMARY = os.path.join(ROOT, "profiles", "grouped_gemm_dram_traffic.txt")
GEMM_SOURCE = os.path.join(ROOT, "paper_1701_06538_b200", "csrc", "ffn_tc.cu")


def ncu_traffic_bytes_per_step(workload_name):
    """The captured DRAM bytes per step of the expert GEMMs for this workload, or None if there is no capture or the
    GEMM source has changed since it was taken."""
    import hashlib
    import re
    try:
        text = open(TRAFFIC_SUMMARY).read()
        sha = hashlib.sha256(open(GEMM_SOURCE, "rb").read()).hexdigest()
    except OSError:
        return None
    m = re.search(r"^ffn_tc_sha256:\s*([0-9a-f]{64})", text, re.M)
    if not m or m.group(1) != sha:
        return None
    m = re.search(r"^traffic_bytes_per_step\[%s\]:\s*([0-9.eE+]+)" % re.escape(workload_name), text, re.M)
    return float(m.group(1)) if m else None


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            with open(path) as f:
                p = json.load(f)
            return {k: float(p[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ------------------------------------------------------------------------------------------ CPU oracle arm
def sample_workload(w, Ts):
    return synth.Workload(**{**w.__dict__, "T": min(Ts, w.T), "name": f"{w.name}[first {min(Ts, w.T)} tokens]"})


def oracle_step(ws, I):
    """One forward+backward of the CPU oracle (test infrastructure) on host arrays."""
    from oracle import moe_oracle as O
    prec = "bf16" if ws.act == "bf16" else "f32"
    F = O.forward(I["x"], I["Wg"], I["Wnoise"], I["noise"], I["W1"], I["b1"], I["W2"], I["b2"], ws.k,
                  ws.w_importance, ws.w_load, prec, hier=ws.hier)
    O.backward(I["dY"], I["x"], I["Wg"], I["Wnoise"], I["noise"], I["W1"], I["b1"], I["W2"], I["b2"], F,
               ws.w_importance, ws.w_load, prec, hier=ws.hier)


def host_inputs_sample(w, Ts, experts=None):
    """Inputs of the first Ts tokens of workload w (the streams are per tensor, so rows [0, Ts) of the
    full tensors are drawn by drawing the full x / noise / dY; expert weights are per expert)."""
    ws = sample_workload(w, Ts)
    x, dY = synth.make_x(w)[:ws.T], synth.make_dY(w)[:ws.T]
    Wg, Wn, noise = synth.make_gate(w)
    noise = tuple(p[:ws.T] for p in noise) if isinstance(noise, tuple) else noise[:ws.T]
    W1, b1, W2, b2 = experts if experts is not None else synth.make_experts(w)
    return ws, dict(x=x, dY=dY, Wg=Wg, Wnoise=Wn, noise=noise, W1=W1, b1=b1, W2=W2, b2=b2)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        return max(n) if n else 1
    except Exception:
        return os.cpu_count() or 1


def cpu_sample_tokens(w, steps):
    """Tokens of the CPU sample. ONE size for both places the oracle is timed (the cpu_baseline of the GPU arm: one
    forward+backward; the --impl reference arm: `steps` of them), because the oracle's rate depends on it (every step
    touches all experts' weights, however few rows an expert gets): about 2e12 flop (10-30 s) per forward+backward, less
    when `steps` of them would not fit in about four minutes, in multiples of 1024 tokens."""
    per_token_flop = 12.0 * w.k * w.d * w.h + 12.0 * w.d * (w.n if w.a == 0 else w.a + w.k1 * w.b)
    budget = min(2.0e12, 1.6e13 / (steps + 1))  # the oracle sustains roughly 1e11 flop/s on these hosts
    return int(max(256, min(w.T, 1024 * int(budget / per_token_flop / 1024))))


def run_reference(args, w):
    rank, _, world = dist_env()
    if rank != 0:
        return
    Ts = cpu_sample_tokens(w, args.steps)
    ws, I = host_inputs_sample(w, Ts)
    for _ in range(min(args.warmup, 1)):
        oracle_step(ws, I)
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        oracle_step(ws, I)
        times.append(time.perf_counter() - t0)
    total = sum(times)
    value = ws.T * args.steps / total
    cores = blas_threads()
    sample = (f"first {ws.T} of {w.T} tokens of {w.name}, all {w.n} experts resident, forward+backward per step "
              f"(the same sample size as the cpu_baseline of the GPU arm at --steps {args.steps})")
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": workload_config(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------ GPU arm
def workload_config(w):
    esz = 2 if w.act == "bf16" else 4
    resident = w.T * w.d * esz * 2 + w.R * (2 * w.d + w.h) * esz + 2 * w.n * w.d * w.h * esz
    return {"workload": w.name, "T": w.T, "d_model": w.d, "hidden": w.h, "experts": w.n, "k": w.k,
            "hierarchical": [w.a, w.k1, w.b, w.k2] if w.a else None, "act": w.act, "gating": "f32",
            "l2": "inputs larger than L2" if resident > 2 * L2_BYTES else "L2 flushed between timed steps",
            "parallelism": "replicas (one per GPU, no collective)"}


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.path = tempfile.mktemp(prefix="clocks_", suffix=".csv")
        self.proc = None
        try:
            self.out = open(self.path, "w")
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(gpu_index)], stdout=self.out,
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.out.close()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        with open(self.path) as f:
            for line in f:
                parts = [p.strip() for p in line.split(",")]
                if len(parts) < 9:
                    continue
                try:
                    sm.append(float(parts[1])); mx.append(float(parts[2])); power.append(float(parts[3]))
                except ValueError:
                    continue
                for name, val in zip(names, parts[5:9]):
                    if val.lower().startswith("active"):
                        reasons.add(name)
        os.unlink(self.path)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


def build_device_state(w, keep_host_experts):
    """Device tensors of the workload. Expert weights are drawn per expert on host threads and moved
    expert by expert, so the host never holds more than a few experts unless the CPU baseline needs them."""
    from paper_1701_06538_b200 import binding as B
    adt = torch.bfloat16 if w.act == "bf16" else torch.float32
    cfg = B.make_config(w.T, w.d, w.h, w.n, w.k, w.act, w.w_importance, w.w_load, w.a, w.k1, w.b, w.k2)
    S = B.moe_query_sizes(cfg)

    def cat(parts):
        if isinstance(parts, tuple):
            return np.concatenate([p.reshape(-1) for p in parts])
        return parts.reshape(-1)

    host = {"x": synth.make_x(w), "dY": synth.make_dY(w)}
    Wg, Wn, noise = synth.make_gate(w)
    host.update(Wg=Wg, Wnoise=Wn, noise=noise)
    D = {"x": torch.from_numpy(host["x"]).to(adt).cuda(), "dY": torch.from_numpy(host["dY"]).to(adt).cuda(),
         "Wg": torch.from_numpy(cat(Wg)).cuda(), "Wnoise": torch.from_numpy(cat(Wn)).cuda(),
         "noise": torch.from_numpy(cat(noise)).cuda()}
    D["W1"] = torch.empty(w.n, w.d, w.h, dtype=adt, device="cuda")
    D["W2"] = torch.empty(w.n, w.h, w.d, dtype=adt, device="cuda")
    D["b1"] = torch.empty(w.n, w.h, dtype=adt, device="cuda")
    D["b2"] = torch.empty(w.n, w.d, dtype=adt, device="cuda")
    if keep_host_experts:
        host["W1"] = np.empty((w.n, w.d, w.h), np.float32); host["W2"] = np.empty((w.n, w.h, w.d), np.float32)
        host["b1"] = np.empty((w.n, w.h), np.float32); host["b2"] = np.empty((w.n, w.d), np.float32)
    with concurrent.futures.ThreadPoolExecutor(max_workers=min(8, os.cpu_count() or 1)) as pool:
        for e, (W1, b1, W2, b2) in enumerate(pool.map(lambda e: synth.make_expert(w, e), range(w.n))):
            D["W1"][e].copy_(torch.from_numpy(W1)); D["W2"][e].copy_(torch.from_numpy(W2))
            D["b1"][e].copy_(torch.from_numpy(b1)); D["b2"][e].copy_(torch.from_numpy(b2))
            if keep_host_experts:
                host["W1"][e], host["b1"][e], host["W2"][e], host["b2"][e] = W1, b1, W2, b2
    e = lambda *s, dt=torch.float32: torch.empty(*s, dtype=dt, device="cuda")
    D.update(y=e(w.T, w.d, dt=adt), losses=e(2), importance=e(w.n), load=e(S.load_elems),
             counts=e(w.n, dt=torch.int32), dX=e(w.T, w.d, dt=adt), dWg=e(S.wg_elems), dWnoise=e(S.wg_elems),
             dW1=e(w.n, w.d, w.h, dt=adt), db1=e(w.n, w.h, dt=adt), dW2=e(w.n, w.h, w.d, dt=adt),
             db2=e(w.n, w.d, dt=adt), ctx=B.empty_bytes(S.ctx_bytes),
             ws=B.empty_bytes(max(S.ws_fwd_bytes, S.ws_bwd_bytes)))
    return cfg, S, D, host


def run_ours(args, w):
    from paper_1701_06538_b200 import binding as B
    rank, local_rank, world = dist_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local_rank)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    peaks, peak_kind = load_peaks()
    want_cpu = rank == 0 and world == 1 and not args.no_cpu_baseline
    cfg, S, D, host = build_device_state(w, keep_host_experts=want_cpu)

    def fwd():
        B.moe_forward(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"], D["y"],
                      D["losses"], D["importance"], D["load"], D["counts"], D["ctx"], D["ws"])

    def bwd():
        B.moe_backward(cfg, D["dY"], D["x"], D["Wg"], D["Wnoise"], D["noise"], D["W1"], D["b1"], D["W2"], D["b2"],
                       D["ctx"], D["dX"], D["dWg"], D["dWnoise"], D["dW1"], D["db1"], D["dW2"], D["db2"], D["ws"])

    small = "flushed" in workload_config(w)["l2"]
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if small else None

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            torch.distributed.barrier()
            torch.cuda.synchronize()

    def timed(step_fn, K):
        """K steps, each between its own pair of events on the launching stream; returns per-step ms."""
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        barrier()
        for a, b in ev:
            if flush_buf is not None:
                flush_buf.fill_(1)
            a.record()
            step_fn()
            b.record()
        barrier()
        return [a.elapsed_time(b) for a, b in ev]

    def step():
        fwd()
        bwd()

    for _ in range(max(args.warmup, 3)):
        step()
    assert B.moe_check_status(D["ws"]) == 0
    # The two library calls only enqueue work on the caller's stream, so the step is captured once in a CUDA graph and
    # replayed (the same kernels, same arguments). Small workloads are bound by the launches outright; at the largest
    # one the gaps between its 51 launches still cost 1.6 % (13.58 ms launched one by one, 13.36 ms replayed, same box).
    graph = None
    if args.graph in ("on", "auto"):
        lc0 = B.moe_debug_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        per_step = B.moe_debug_launch_count() - lc0
        for _ in range(3):
            graph.replay()
        torch.cuda.synchronize()
        assert B.moe_check_status(D["ws"]) == 0
    sampler = ClockSampler(local_rank)
    l0 = B.moe_debug_launch_count()
    ms = timed(graph.replay if graph else step, args.steps)
    launches = per_step * args.steps if graph else B.moe_debug_launch_count() - l0

    # end to end: every step copies its inputs (x, noise, dY) from pinned host memory and copies its results
    # (y, dX, losses) back, all inside the timed region. Three streams and three sets of device buffers let the
    # copies of neighbouring steps overlap the kernels of the current one; the kernels themselves are the
    # same calls in the same order as in the device-resident measurement.
    hx, hdY = torch.from_numpy(host["x"]).to(D["x"].dtype).pin_memory(), torch.from_numpy(host["dY"]).to(D["x"].dtype).pin_memory()
    hnoise = D["noise"].cpu().pin_memory()
    hy, hdX, hl = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory(), torch.empty(2).pin_memory()
    NSETS = 3  # with two, the 0.6 GB of inputs of step i + 2 had one step's time to arrive: as long as the copy itself
    bufs = [{k: (D[k] if b == 0 else torch.empty_like(D[k])) for k in ("x", "noise", "dY", "y", "dX", "losses")}
            for b in range(NSETS)]
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()

    def e2e_fwd(Bf):
        B.moe_forward(cfg, Bf["x"], D["Wg"], D["Wnoise"], Bf["noise"], D["W1"], D["b1"], D["W2"], D["b2"],
                      Bf["y"], Bf["losses"], D["importance"], D["load"], D["counts"], D["ctx"], D["ws"])

    def e2e_bwd(Bf):
        B.moe_backward(cfg, Bf["dY"], Bf["x"], D["Wg"], D["Wnoise"], Bf["noise"], D["W1"], D["b1"], D["W2"],
                       D["b2"], D["ctx"], Bf["dX"], D["dWg"], D["dWnoise"], D["dW1"], D["db1"], D["dW2"],
                       D["db2"], D["ws"])

    # the two calls of a step as one graph each per buffer set (the copies and the events between them stay outside)
    e2e_graphs = None
    if graph is not None:
        e2e_graphs = []
        for Bf in bufs:
            gf, gb = torch.cuda.CUDAGraph(), torch.cuda.CUDAGraph()
            with torch.cuda.graph(gf, stream=s_comp):
                e2e_fwd(Bf)
            with torch.cuda.graph(gb, stream=s_comp):
                e2e_bwd(Bf)
            e2e_graphs.append((gf, gb))
        torch.cuda.synchronize()

    def run_e2e(K):
        ev_in_f = [torch.cuda.Event() for _ in range(K)]   # x and noise of step i are on the device
        ev_in_b = [torch.cuda.Event() for _ in range(K)]   # dY too
        ev_fwd = [torch.cuda.Event() for _ in range(K)]
        ev_comp = [torch.cuda.Event() for _ in range(K)]
        ev_out = [torch.cuda.Event() for _ in range(K)]
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        with torch.cuda.stream(s_in):
            t0.record()
        for i in range(K):
            Bf = bufs[i % NSETS]
            with torch.cuda.stream(s_in):
                if i >= NSETS:
                    s_in.wait_event(ev_comp[i - NSETS])  # the kernels that read this input set are done
                Bf["x"].copy_(hx, non_blocking=True); Bf["noise"].copy_(hnoise, non_blocking=True)
                ev_in_f[i].record()
                Bf["dY"].copy_(hdY, non_blocking=True)  # only the backward needs it: it arrives during the forward
                ev_in_b[i].record()
            with torch.cuda.stream(s_comp):
                s_comp.wait_event(ev_in_f[i])
                if i >= NSETS:
                    s_comp.wait_event(ev_out[i - NSETS])  # this output set has been copied out
                if e2e_graphs: e2e_graphs[i % NSETS][0].replay()
                else: e2e_fwd(Bf)
                ev_fwd[i].record()
                s_comp.wait_event(ev_in_b[i])
                if e2e_graphs: e2e_graphs[i % NSETS][1].replay()
                else: e2e_bwd(Bf)
                ev_comp[i].record()
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_fwd[i])  # y and the losses leave while the backward runs
                hy.copy_(Bf["y"], non_blocking=True); hl.copy_(Bf["losses"], non_blocking=True)
                s_out.wait_event(ev_comp[i])
                hdX.copy_(Bf["dX"], non_blocking=True)
                ev_out[i].record()
        with torch.cuda.stream(s_out):
            t1.record()
        barrier()
        return t0.elapsed_time(t1)

    run_e2e(2)
    ms_e2e = [run_e2e(args.steps)]
    clocks = sampler.stop()
    h2d = hx.numel() * hx.element_size() * 2 + hnoise.numel() * 4
    d2h = hy.numel() * hy.element_size() * 2 + 8

    total_ms, total_e2e = replicas.max_over_ranks([sum(ms), sum(ms_e2e)], device="cuda")
    value = replicas.job_throughput(w.T, args.steps, total_ms, world)
    value_e2e = replicas.job_throughput(w.T, args.steps, total_e2e, world)

    stages = stage_timings(B, cfg, S, D, w, (lambda: flush_buf.fill_(1)) if flush_buf is not None else (lambda: None),
                           max(3, min(args.steps, 10)), peaks)
    # Roofline of the dominant kernel family, the expert grouped GEMMs (six launches per step). They are bound by the
    # tensor cores when the segments are long and by HBM when there are so many experts that every weight is read
    # for a handful of rows (c4): both fractions are computed from the algorithmic flop / bytes, the larger one binds.
    esz = 2 if w.act == "bf16" else 4
    gemm_flop = 12.0 * w.R * w.d * w.h
    gemm_bytes = (6 * w.R * w.d + 5 * w.R * w.h) * esz + 6 * w.n * w.d * w.h * esz
    gemm_ms = stages["expert_ffn"]["ms"] + stages["expert_ffn_bwd"]["ms"]
    achieved = gemm_flop / (gemm_ms / 1e3) / 1e12
    achieved_gbs = gemm_bytes / (gemm_ms / 1e3) / 1e9
    traffic = ncu_traffic_bytes_per_step(workload_config(w)["workload"])
    kernel = "expert grouped GEMMs (moe_expert_ffn + moe_expert_ffn_bwd, 6 launches; achieved = per-step flop or bytes / per-step time)"
    if w.act != "bf16":
        roof = {"bound": "alu", "kernel": "expert grouped GEMMs, fp32 SIMT", "achieved": achieved,
                "peak": FP32_PEAK_TFLOPS, "unit": "TFLOP/s", "frac": achieved / FP32_PEAK_TFLOPS, "traffic": None,
                "peak_kind": "derived: 148 SMs x 128 FP32 lanes x 2 x 1.965 GHz"}
    elif achieved_gbs / peaks["hbm_gbs"] > achieved / peaks["bf16_tflops"]:
        roof = {"bound": "hbm", "kernel": kernel, "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": achieved_gbs / peaks["hbm_gbs"], "traffic": traffic,
                "peak_kind": f"{peak_kind} copy bandwidth", "tensor_tflops": achieved}
    else:
        # the stage timers run a few launches back to back (about 0.1 s), not a seconds-long loop under the power cap:
        # the burst figure is the denominator; the sustained and the nominal one are printed beside it
        roof = {"bound": "tensor", "kernel": kernel, "achieved": achieved, "peak": peaks["bf16_tflops"],
                "unit": "TFLOP/s", "frac": achieved / peaks["bf16_tflops"], "traffic": traffic,
                "peak_kind": f"{peak_kind} burst bf16 (cuBLAS, best of 10)",
                "frac_of_burst": achieved / peaks["bf16_tflops"],
                "frac_of_sustained": achieved / peaks["bf16_tflops_sustained"],
                "frac_of_nominal_2250": achieved / 2250.0, "algorithmic_bytes": gemm_bytes,
                "forward_tflops": 4.0 * w.R * w.d * w.h / stages["expert_ffn"]["ms"] / 1e9,
                "backward_tflops": 8.0 * w.R * w.d * w.h / stages["expert_ffn_bwd"]["ms"] / 1e9}

    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
           "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "bf16" if w.act == "bf16" else "f32",
           "data": "synthetic", "config": dict(workload_config(w), launch="cuda graph replay" if graph else "stream"),
           "clocks": clocks,
           "e2e": {"value": value_e2e, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                   "ms_per_step": total_e2e / args.steps},
           "gpu_launches": launches, "roofline": roof, "stages": stages,
           "balance": balance_metrics(D)}
    if want_cpu:
        Ts = cpu_sample_tokens(w, args.steps)
        wsamp, I = host_inputs_sample(w, Ts, experts=(host["W1"], host["b1"], host["W2"], host["b2"]))
        t0 = time.perf_counter()
        oracle_step(wsamp, I)
        sec = time.perf_counter() - t0
        out["cpu_baseline"] = {"value": wsamp.T / sec, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                               "sample": f"first {wsamp.T} of {w.T} tokens, all {w.n} experts, one forward+backward "
                                         f"({sec:.1f} s); --impl reference uses the same sample size at --steps {args.steps}"}
    if rank == 0:
        print(json.dumps(out))
    if world > 1:
        torch.distributed.destroy_process_group()


def run_balanced(args, w):
    """The same layer with strictly balanced gating (Appendix F): every expert receives exactly k T / n examples, so
    the grouped GEMMs run on uniform segments. One step = gate, dispatch, experts, combine and their backward, composed
    from the stage calls of the C ABI. Second workload of the library; the headline line is the noisy top-k one."""
    from paper_1701_06538_b200 import binding as B
    rank, local_rank, world = dist_env()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local_rank)
    peaks, peak_kind = load_peaks()
    cfg, S, D, host = build_device_state(w, keep_host_experts=False)
    Sb = B.moe_query_balanced_sizes(cfg)
    T, d, h, n, k, R = w.T, w.d, w.h, w.n, w.k, w.R
    adt = D["x"].dtype
    e = lambda *s_, dt=torch.float32: torch.empty(*s_, dtype=dt, device="cuda")
    thr = torch.full((n,), 1.0 / n, device="cuda")
    G = dict(logits=e(T, n), probs=e(T, n), mask_bits=e(T, Sb.mask_words, dt=torch.int32), tok_of_row=e(R, dt=torch.int32),
             offsets=e(n + 1, dt=torch.int32), den=e(T), tok_ptr=e(T + 1, dt=torch.int32), tok_rows=e(R, dt=torch.int32),
             loss=e(1), thr_counts=e(n, dt=torch.int32), ws=B.empty_bytes(Sb.ws_bytes))
    xs, hid, ys, dys, dxs = e(R, d, dt=adt), e(R, h, dt=adt), e(R, d, dt=adt), e(R, d, dt=adt), e(R, d, dt=adt)
    dG_row, dWg, dXg, dthr = e(R), e(d, n), e(T, d), e(n)
    Wg = D["Wg"][:d * n]
    calls = {
        "gate_balanced": lambda: B.moe_gate_balanced(cfg, D["x"], Wg, thr, G["logits"], G["probs"], G["mask_bits"],
                                                     G["tok_of_row"], G["offsets"], G["den"], G["tok_ptr"], G["tok_rows"],
                                                     G["loss"], G["thr_counts"], G["ws"]),
        "dispatch_balanced": lambda: B.moe_dispatch_balanced(cfg, D["x"], G["tok_of_row"], xs),
        "expert_ffn": lambda: B.moe_expert_ffn(cfg, xs, G["offsets"], D["W1"], D["b1"], D["W2"], D["b2"], hid, ys, D["ws"]),
        "combine_balanced": lambda: B.moe_combine_balanced(cfg, ys, G["probs"], G["den"], G["tok_ptr"], G["tok_rows"], D["y"]),
        "combine_balanced_bwd": lambda: B.moe_combine_balanced_bwd(cfg, D["dY"], ys, G["probs"], G["den"], G["tok_of_row"],
                                                                   dG_row, dys),
        "expert_ffn_bwd": lambda: B.moe_expert_ffn_bwd(cfg, xs, hid, dys, G["offsets"], D["W1"], D["W2"], dxs, D["dW1"],
                                                       D["db1"], D["dW2"], D["db2"], D["ws"]),
        "gate_balanced_bwd": lambda: B.moe_gate_balanced_bwd(cfg, D["x"], Wg, G["probs"], G["mask_bits"], G["den"], thr,
                                                             G["tok_ptr"], G["tok_rows"], dG_row, G["thr_counts"], 1.0, dWg,
                                                             dXg, dthr, G["ws"]),
        "dispatch_balanced_bwd": lambda: B.moe_dispatch_balanced_bwd(cfg, dxs, G["tok_ptr"], G["tok_rows"], dXg, D["dX"]),
    }

    def step():
        for fn in calls.values():
            fn()

    small = "flushed" in workload_config(w)["l2"]
    flush_buf = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device="cuda") if small else None

    def timed(fn, K):
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
        torch.cuda.synchronize()
        for a, b in ev:
            if flush_buf is not None:
                flush_buf.fill_(1)
            a.record(); fn(); b.record()
        torch.cuda.synchronize()
        return [a.elapsed_time(b) for a, b in ev]

    for _ in range(max(args.warmup, 3)):
        step()
    assert B.moe_check_status(D["ws"]) == 0
    sampler = ClockSampler(local_rank)
    l0 = B.moe_debug_launch_count()
    ms = timed(step, args.steps)
    launches = B.moe_debug_launch_count() - l0
    hx, hdY = D["x"].cpu().pin_memory(), D["dY"].cpu().pin_memory()
    hy, hdX = torch.empty_like(hx).pin_memory(), torch.empty_like(hx).pin_memory()

    def e2e_step():
        D["x"].copy_(hx, non_blocking=True); D["dY"].copy_(hdY, non_blocking=True)
        step()
        hy.copy_(D["y"], non_blocking=True); hdX.copy_(D["dX"], non_blocking=True)

    e2e_step()
    ms_e2e = timed(e2e_step, args.steps)
    clocks = sampler.stop()
    stages = {name: {"ms": statistics.mean(timed(fn, max(3, min(args.steps, 10))))} for name, fn in calls.items()}
    esz = 2 if w.act == "bf16" else 4
    gemm_ms = stages["expert_ffn"]["ms"] + stages["expert_ffn_bwd"]["ms"]
    achieved = 12.0 * R * d * h / (gemm_ms / 1e3) / 1e12
    gemm_bytes = (6 * R * d + 5 * R * h) * esz + 6 * n * d * h * esz
    achieved_gbs = gemm_bytes / (gemm_ms / 1e3) / 1e9
    hbm_bound = achieved_gbs / peaks["hbm_gbs"] > achieved / peaks["bf16_tflops"]
    roof = {"bound": "hbm" if hbm_bound else "tensor", "kernel": "expert grouped GEMMs on uniform segments (6 launches)",
            "achieved": achieved_gbs if hbm_bound else achieved, "peak": peaks["hbm_gbs"] if hbm_bound else peaks["bf16_tflops"],
            "unit": "GB/s" if hbm_bound else "TFLOP/s",
            "frac": achieved_gbs / peaks["hbm_gbs"] if hbm_bound else achieved / peaks["bf16_tflops"], "traffic": None,
            "peak_kind": f"{peak_kind} " + ("copy bandwidth" if hbm_bound else "burst bf16"), "tensor_tflops": achieved}
    counts = torch.diff(G["offsets"]).cpu()
    print(json.dumps({
        "metric": METRIC, "value": T * args.steps / (sum(ms) / 1e3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": sum(ms) / args.steps, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16" if w.act == "bf16" else "f32", "data": "synthetic",
        "config": dict(workload_config(w), gating="strictly balanced (Appendix F): every expert gets exactly k T / n rows",
                       rows_per_expert=int(Sb.m), launch="stream"),
        "clocks": clocks,
        "e2e": {"value": T * args.steps / (sum(ms_e2e) / 1e3), "unit": UNIT, "h2d_bytes_per_step": 2 * hx.numel() * esz,
                "d2h_bytes_per_step": 2 * hx.numel() * esz, "ms_per_step": sum(ms_e2e) / args.steps},
        "gpu_launches": launches, "roofline": roof, "stages": stages,
        "balance": {"rows_per_expert_min": int(counts.min()), "rows_per_expert_max": int(counts.max()),
                    "examples_without_expert": int((torch.diff(G["tok_ptr"]) == 0).sum()),
                    "loss_batchwise": float(G["loss"][0])}}))


def balance_metrics(D):
    """The balance metrics of the paper's loss-ablation table, for the realised routing."""
    imp, load, counts = D["importance"].double(), D["load"][:D["importance"].numel()].double(), D["counts"].double()
    cv = lambda v: float(v.std(unbiased=False) / v.mean())
    return {"cv_importance": cv(imp), "cv_load": cv(load), "max_over_mean_load": float(load.max() / load.mean()),
            "max_over_min_count": float(counts.max() / counts.min().clamp(min=1)),
            "max_over_mean_count": float(counts.max() / counts.mean())}


def stage_timings(B, cfg, S, D, w, flush, K, peaks):
    """Each stage call alone, K launches between events, on the tensors the fused forward saved."""
    V = B.ctx_views(cfg, D["ctx"])
    T, d, h, n, k, R = w.T, w.d, w.h, w.n, w.k, w.R
    esz = 2 if w.act == "bf16" else 4
    adt = D["x"].dtype
    e = lambda *s, dt=torch.float32: torch.empty(*s, dtype=dt, device="cuda")
    ws = D["ws"]
    dgates, dys, dxs = e(S.gates_elems), e(R, d, dt=adt), e(R, d, dt=adt)
    dload, dXe, dXg = e(S.dload_elems), e(T, d), e(T, d)
    gate_cols = S.gate_cols
    calls = {
        "gate": (lambda: B.moe_gate(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], V["topk_idx"], V["gates"],
                                    V["clean"], V["raw_noise"], V["kth_vals"], V["kth_idx"], ws),
                 4.0 * T * d * gate_cols, T * d * esz + 3 * 4 * T * gate_cols + 8 * R + 16 * T),
        "dispatch": (lambda: B.moe_dispatch(cfg, D["x"], V["topk_idx"], V["xs"], V["perm"], V["inv_perm"],
                                            V["counts"], V["offsets"], ws), 0.0, (1 + k) * T * d * esz + 12 * R),
        "expert_ffn": ((lambda: B.moe_expert_ffn_bits(cfg, V["xs"], V["offsets"], D["W1"], D["b1"], D["W2"], D["b2"],
                                                      V["hid"], V["ys"], V["relu_bits"], ws)) if "relu_bits" in V else
                       (lambda: B.moe_expert_ffn(cfg, V["xs"], V["offsets"], D["W1"], D["b1"], D["W2"], D["b2"],
                                                 V["hid"], V["ys"], ws)),
                       4.0 * R * d * h, (2 * R * d + 2 * R * h) * esz + 2 * n * d * h * esz),
        "combine": (lambda: B.moe_combine(cfg, V["ys"], V["gates"], V["inv_perm"], D["y"]), 0.0,
                    (k + 1) * T * d * esz + 8 * R),
        "losses": (lambda: B.moe_losses(cfg, V["topk_idx"], V["gates"], V["clean"], V["raw_noise"], V["kth_vals"],
                                        D["importance"], D["load"], D["losses"], ws), 0.0, 2 * 4 * T * gate_cols + 16 * R),
        "combine_bwd": (lambda: B.moe_combine_bwd(cfg, D["dY"], V["ys"], V["gates"], V["inv_perm"], dgates, dys), 0.0,
                        (1 + 2 * k) * T * d * esz + 12 * R),
        # the calls the fused path makes: with the ReLU mask as bits where the layer runs on the tensor cores
        "expert_ffn_bwd": ((lambda: B.moe_expert_ffn_bwd_bits(cfg, V["xs"], V["hid"], V["relu_bits"], dys, V["offsets"],
                                                              D["W1"], D["W2"], dxs, D["dW1"], D["db1"], D["dW2"],
                                                              D["db2"], ws)) if "relu_bits" in V else
                           (lambda: B.moe_expert_ffn_bwd(cfg, V["xs"], V["hid"], dys, V["offsets"], D["W1"], D["W2"],
                                                         dxs, D["dW1"], D["db1"], D["dW2"], D["db2"], ws)),
                           8.0 * R * d * h, (4 * R * d + 3 * R * h) * esz + 4 * n * d * h * esz),
        "losses_bwd": (lambda: B.moe_losses_bwd(cfg, D["importance"], D["load"], V["topk_idx"], dgates, dload, ws),
                       0.0, 12 * R),
        "gate_bwd": (lambda: B.moe_gate_bwd(cfg, D["x"], D["Wg"], D["Wnoise"], D["noise"], V["clean"], V["raw_noise"],
                                            V["topk_idx"], V["gates"], V["kth_vals"], V["kth_idx"], dgates, dload,
                                            D["dWg"], D["dWnoise"], dXg, ws),
                     8.0 * T * d * gate_cols, T * d * (esz + 4) + 5 * 4 * T * gate_cols),
        "dispatch_bwd": (lambda: B.moe_dispatch_bwd(cfg, dxs, V["inv_perm"], dXe), 0.0, k * T * d * esz + T * d * 4),
    }
    if d % 8 == 0:
        # the layer as it sits in the paper's models (sigmoid, dropout, residual fused into the combine kernels): timed
        # beside the plain stages, not part of the step; the keep mask is one bit per activation
        keep = torch.from_numpy(synth.make_keep_bits(w, 0.3)).cuda()
        out_layer = e(T, d, dt=adt)
        calls["combine_layer"] = (lambda: B.moe_combine_layer(cfg, V["ys"], V["gates"], V["inv_perm"], D["x"], keep, 0.3,
                                                              out_layer), 0.0, (k + 2) * T * d * esz + T * d // 8 + 8 * R)
        calls["combine_layer_bwd"] = (lambda: B.moe_combine_layer_bwd(cfg, D["dY"], V["ys"], V["gates"], V["inv_perm"],
                                                                      keep, 0.3, dgates, dys), 0.0,
                                      (1 + 2 * k) * T * d * esz + T * d // 8 + 12 * R)
    # the optimiser step of the paper's large models (factored second-moment Adam, beta1 = 0) on the expert parameters:
    # timed beside the stages, not part of the step; learning rate 0 leaves the weights as they are
    adam_state = torch.zeros(S.adam_state_elems, device="cuda")
    adam_ws = B.empty_bytes(S.ws_adam_bytes)
    calls["adam_factored"] = (lambda: B.moe_expert_adam_factored(cfg, D["W1"], D["b1"], D["W2"], D["b2"], D["dW1"], D["db1"],
                                                                 D["dW2"], D["db2"], adam_state, 0.0, 0.999, 1e-8, 1, adam_ws),
                              0.0, 4 * 2 * n * d * h * esz)
    # Every stage between its own pair of events, the stages taken in turn K times over (not K launches of one stage
    # back to back): the chip then sits in the power and clock state of a real step, where tensor-core and streaming
    # kernels alternate, instead of the state ten identical GEMM launches in a row drive it into.
    for fn, _, _ in calls.values():
        fn()
    torch.cuda.synchronize()
    ev = {name: [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
          for name in calls}
    for i in range(K):
        for name, (fn, _, _) in calls.items():
            a, b = ev[name][i]
            flush()  # small workloads: L2 written over before every timed call
            a.record()
            fn()
            b.record()
    torch.cuda.synchronize()
    out = {}
    for name, (fn, flop, byts) in calls.items():
        ms = statistics.mean(a.elapsed_time(b) for a, b in ev[name])
        rec = {"ms": ms, "GB/s": byts / ms / 1e6, "hbm_frac": byts / ms / 1e6 / peaks["hbm_gbs"]}
        if flop:
            rec["TFLOP/s"] = flop / ms / 1e9
        out[name] = rec
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="c5", choices=sorted(synth.CONFIGS))
    ap.add_argument("--tokens", type=int, default=0, help="override T (smaller captures under a profiler)")
    ap.add_argument("--graph", default="auto", choices=["auto", "on", "off"],
                    help="replay the step from a CUDA graph (auto = on; off: launch kernel by kernel)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--gating", default="noisy-topk", choices=["noisy-topk", "balanced"],
                    help="balanced: the strictly balanced gating of Appendix F (flat configs whose k T is a multiple of n)")
    args = ap.parse_args()
    w = synth.CONFIGS[args.config]
    if args.tokens:
        w = w.scaled(args.tokens)
    if args.gating == "balanced" and args.impl == "ours":
        run_balanced(args, w)
    elif args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()

"""Benchmark of the DMTD decode path: generated tokens/s on a Qwen3-4B-shaped model.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl native|reference]
                    [--workload qwen3_4b_b1|qwen3_4b_b32|...] [--tau T]

A step is one steady-state decode cycle (Section 2.2 of the paper): one full pass (refill of
the lower layers + newest token through all layers) and tau-1 passes through the decoding
layers only, i.e. tau tokens per sequence.  Weights and prompts are seeded synthetic data of
the workload's shape.  Rank 0 prints one JSON line.
"""
import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from synthetic import SHAPES, WORKLOADS, make_prompts, make_weights, weight_bytes  # noqa: E402

METRIC = "generated tokens/s (decode, steady-state DMTD cycles)"
UNIT = "tokens/s"


def bytes_per_cycle(shape, L_d, tau, batch, mean_ctx, kv_bytes=2):
    """Bytes the cycle must move: every layer-pass reads that layer's weights once and the KV
    of every sequence once; every pass reads the tied head once."""
    w_layer, w_head = weight_bytes(shape)
    layer_passes = shape.n_layers + (tau - 1) * L_d
    kv_per_pos = 2 * shape.n_kv_heads * shape.head_dim * kv_bytes   # K and V
    return layer_passes * w_layer + tau * w_head + layer_passes * batch * mean_ctx * kv_per_pos


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.samples, self.reasons, self.max_mhz, self._halt = [], set(), None, threading.Event()
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksThrottleReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksThrottleReasonHwThermalSlowdown: "hw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksThrottleReasonSwPowerCap: "sw_power_cap"}
        while not self._halt.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for bit, name in names.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(s)}


def physical_gpu_index(local):
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local])
        except Exception:
            return local
    return local


def host_copy(weights):
    return {"embed": weights["embed"].cpu(), "final_norm": weights["final_norm"].cpu(),
            "layers": [{k: v.cpu() for k, v in lw.items()} for lw in weights["layers"]]}


def time_oracle(shape, weights_host, L_d, tau, steps, warmup, prompt_len=8):
    """The CPU oracle as it stands, on this machine's host cores: `steps` decode cycles of one
    sequence after a short prompt.  Returns (tokens/s, per-step seconds, cores used)."""
    import oracle
    cores = torch.get_num_threads()
    try:
        cores = len(os.sched_getaffinity(0))
    except Exception:
        pass
    o = oracle.Oracle(shape, weights_host, L_d=L_d, tau=tau, max_batch=1,
                      max_seq=prompt_len + (steps + warmup + 2) * tau + 2)
    prompt = make_prompts(shape.vocab, 1, prompt_len, seed=1).numpy()
    o.prefill(prompt, want_logits=False)
    if tau > 1:
        o.decode_cycle(tau, want_logits=False)              # finish cycle 1
    for _ in range(warmup):
        o.decode_cycle(tau, want_logits=False)
    t0 = time.perf_counter()
    for _ in range(steps):
        o.decode_cycle(tau, want_logits=False)
    dt = time.perf_counter() - t0
    return steps * tau / dt, dt / max(steps, 1), cores


def run_reference(args, wl, shape):
    """The reference arm: the oracle timed on the host cores (rank 0 only)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    w = make_weights(shape, seed=wl.weight_seed, device=dev)
    wh = host_copy(w) if dev == "cuda" else w
    del w
    tps, sec_per_step, cores = time_oracle(shape, wh, wl.L_d, args.tau, args.steps, args.warmup)
    sample = (f"{args.steps} decode cycles (tau={args.tau}) of one sequence after an 8-token prompt, "
              f"{args.warmup} warm-up cycles, whole model")
    line = {"impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec_per_step * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic",
            "config": {"workload": wl.name, "shape": wl.shape, "tau": args.tau, "L_d": wl.L_d,
                       "batch": 1, "note": "CPU oracle, bounded sample"},
            "cpu_baseline": {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


# DRAM traffic / algorithmic bytes of the dominant kernel, from ncu captures of exactly the kernel
# and the shape named here (profiles/); any other workload reports traffic = null.
NCU_TRAFFIC_RATIO = {
    # profiles/dmtd_pass_kernel_qwen3_4b_l4_b1_ncu_full.md: the three launches of a cycle on the 4-layer model read
    # and wrote 3.9871 GB for 3.9660 GB of weights and KV; the 36-layer workload runs the same kernel on the same
    # layer and head shapes, and its traffic grows with the bytes streamed
    ("qwen3_4b_l4_b1", "fused"): 1.0053,
    ("qwen3_4b_b1", "fused"): 1.0053,
}


def measure_workload(eng, wl, shape, prompts, tau, K, W, replicas, want_tau1=True):
    """Device-timed decode cycles of one workload on one engine.  Returns a dict with the elapsed
    milliseconds over K cycles, the launch count, the per-cycle times, the context range during
    timing and, if asked, the tokens/s of the same engine at tau = 1."""
    B, P = wl.batch, wl.prompt_len

    def timed_cycles(tau_now, steps, warm):
        eng.prefill(prompts)
        if tau_now > 1:
            eng.decode_cycle(tau_now)
        for _ in range(warm):
            eng.decode_cycle(tau_now)
        out = torch.zeros(B, tau_now, dtype=torch.int32, device="cuda")
        torch.cuda.synchronize()
        replicas.barrier()
        l0 = eng.launch_count()
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(steps + 1)]
        ev[0].record()
        for i in range(steps):
            eng.decode_cycle(tau_now, out_tokens=out)
            ev[i + 1].record()
        torch.cuda.synchronize()
        replicas.barrier()
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(steps)]
        return ev[0].elapsed_time(ev[steps]), eng.launch_count() - l0, per

    ms, launches, per_cycle = timed_cycles(tau, K, W)
    ctx_begin = P + 1 + (tau - 1) + W * tau
    res = {"ms": ms, "launches": launches, "per_cycle": per_cycle, "ctx_begin": ctx_begin,
           "mean_ctx": ctx_begin + K * tau / 2.0, "tau1": None}
    if tau != 1 and want_tau1:
        eng.reset()
        eng.set_tau(1)
        k1 = max(3, min(K, 60))
        ms1, _, _ = timed_cycles(1, k1, W)
        res["tau1"] = B * k1 / (ms1 * 1e-3)
        eng.reset()
        eng.set_tau(tau)
    return res


def roofline_of(shape, wl, tau, res, K, peak, peak_src):
    """The roofline object of one measured workload (see the design doc for the byte model)."""
    kvb = 4 if wl.kv_dtype == "f32" else 2
    cyc_bytes = bytes_per_cycle(shape, wl.L_d, tau, wl.batch, res["mean_ctx"], kv_bytes=kvb)
    cyc_bytes_bf16kv = bytes_per_cycle(shape, wl.L_d, tau, wl.batch, res["mean_ctx"], kv_bytes=2)
    # one launch per pass on the persistent-kernel path: tau launches per cycle (plus a token gather)
    fused = res["launches"] <= K * (tau + 1)
    n_launch = tau if fused else res["launches"] / K
    launch_bytes = cyc_bytes / tau
    launch_s = res["ms"] / K * 1e-3 / tau
    achieved = launch_bytes / launch_s / 1e9
    ratio = NCU_TRAFFIC_RATIO.get((wl.name, "fused" if fused else "per_step"))
    return {"bound": "hbm",
            "kernel": ("dmtd_pass_kernel (one launch per pass; average over the 1 full + tau-1 "
                       "decoding-layer passes of a cycle)") if fused else
                      "per-step kernels (all kernels of 1 full + tau-1 short passes, as one unit)",
            "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "peak_source": peak_src, "frac_of_nominal_8TBs": achieved / 8000.0,
            "bytes_per_cycle": cyc_bytes, "launches_per_cycle": n_launch,
            "algorithmic_bytes_per_launch": launch_bytes, "avg_launch_us": launch_s * 1e6,
            # with the KV cache counted at 2 bytes per value (the byte model's own figure) whatever the cache holds
            "frac_with_bf16_kv_bytes": cyc_bytes_bf16kv / (res["ms"] / K * 1e-3) / 1e9 / peak,
            "traffic": launch_bytes * ratio if ratio else None}


def run_native(args, wl, shape):
    from paper_2510_11958_b200 import Dmtd, replicas
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}"
    torch.cuda.set_device(local)
    if world > 1:
        replicas.init_from_env("nccl")
    tau, L_d, B, P = args.tau, wl.L_d, wl.batch, wl.prompt_len
    K, W = args.steps, args.warmup
    n_tokens_total = 1 + (tau - 1) + (W + K) * tau
    max_seq = P + n_tokens_total + tau + 1
    peaks_path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(peaks_path):
        peak, peak_src = json.load(open(peaks_path))["hbm_gbs"], "measured"
    else:
        peak, peak_src = 6650.0, "fallback"

    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        weights = make_weights(shape, seed=wl.weight_seed, device="cuda")
        wh = host_copy(weights) if (rank == 0 and world == 1 and not args.no_cpu_baseline) else None
        eng = Dmtd(shape, weights, L_d=L_d, tau=tau, max_batch=B, max_seq=max_seq, kv_dtype=wl.kv_dtype)
        for kv in args.option:
            name, value = kv.split("=")
            eng.set_option(name, int(value))
        prompts_host = make_prompts(shape.vocab, B, P, seed=wl.prompt_seed).pin_memory()
        prompts = prompts_host.cuda()
        memory = {k: round(v / 1e9, 3) for k, v in eng.memory_info().items()}

        sampler = ClockSampler(physical_gpu_index(local))
        sampler.start()
        res = measure_workload(eng, wl, shape, prompts, tau, K, W, replicas, want_tau1=False)
        clocks = sampler.stop()
        ms, launches, per_cycle = res["ms"], res["launches"], res["per_cycle"]
        # the same build at tau = 1 (ordinary decoding): DMTD's speedup
        tau1 = None
        if tau != 1 and not args.no_tau1:
            eng.reset()
            eng.set_tau(1)
            k1 = max(3, min(K, 60))
            r1 = measure_workload(eng, wl, shape, prompts, 1, k1, W, replicas, want_tau1=False)
            tau1 = B * k1 / (r1["ms"] * 1e-3)
            eng.reset()
            eng.set_tau(tau)

        # end to end through the host-buffer calls: prompt upload + prefill + every cycle's
        # tokens read back to pinned host memory
        e2e_request = e2e_decode = None
        calls = 1
        if not args.no_e2e:
            eng.reset()
            out_host = torch.zeros(B, tau, dtype=torch.int32).pin_memory()
            gen = 1 + (tau - 1) + K * tau
            torch.cuda.synchronize()
            replicas.barrier()
            t0 = time.perf_counter()
            eng.prefill_host(prompts_host)
            t_prefill = time.perf_counter()
            n_done, calls = 1, 0
            while n_done < gen:
                n_done += eng.decode_cycle_host(gen - n_done, out_host)
                calls += 1
            t1 = time.perf_counter()
            replicas.barrier()
            e2e_request = B * gen / (t1 - t0) * world
            e2e_decode = B * (gen - 1) / (t1 - t_prefill) * world
            e2e_prefill_ms = (t_prefill - t0) * 1e3
            # the prefill as a dense contraction: 2 flop per weight and prompt row in the layers, the causal
            # attention products, the head on the last row; against the measured sustained bf16 rate
            flops = (2.0 * shape.n_layers * shape.params_per_layer * B * P
                     + shape.n_layers * B * 4.0 * shape.n_q_heads * shape.head_dim * P * (P + 1) / 2
                     + 2.0 * shape.vocab * shape.hidden * B)
            tf_peak = None
            if os.path.exists(peaks_path):
                tf_peak = json.load(open(peaks_path)).get("bf16_tflops_sustained")
            prefill = {"ms": e2e_prefill_ms, "tokens_per_s": B * P / (e2e_prefill_ms * 1e-3),
                       "tflops": flops / (e2e_prefill_ms * 1e-3) / 1e12,
                       "frac_of_bf16_sustained": (flops / (e2e_prefill_ms * 1e-3) / 1e12 / tf_peak) if tf_peak else None,
                       "note": "prompt upload + chunked prefill + first token read back, host timed"}

        # the metric's second batch size, in the same run: batch 32 of the same model at the same tau
        bs32 = None
        if args.bs32 and wl.name == "qwen3_4b_b1" and world == 1:
            eng.close()
            del eng
            torch.cuda.empty_cache()
            wl32 = WORKLOADS["qwen3_4b_b32"]
            K32, W32 = args.bs32_steps, 3
            ms32_seq = wl32.prompt_len + 1 + (tau - 1) + (W32 + K32) * tau + tau + 1
            eng32 = Dmtd(shape, weights, L_d=wl32.L_d, tau=tau, max_batch=wl32.batch, max_seq=ms32_seq,
                         kv_dtype=wl32.kv_dtype)
            p32 = make_prompts(shape.vocab, wl32.batch, wl32.prompt_len, seed=wl32.prompt_seed).cuda()
            sampler32 = ClockSampler(physical_gpu_index(local))
            sampler32.start()
            r32 = measure_workload(eng32, wl32, shape, p32, tau, K32, W32, replicas, want_tau1=False)
            clocks32 = sampler32.stop()
            eng32.reset()
            eng32.set_tau(1)
            r32_1 = measure_workload(eng32, wl32, shape, p32, 1, K32, W32, replicas, want_tau1=False)
            tps32 = wl32.batch * tau * K32 / (r32["ms"] * 1e-3)
            tps32_1 = wl32.batch * K32 / (r32_1["ms"] * 1e-3)
            bs32 = {"workload": wl32.name, "value": tps32, "unit": UNIT, "steps": K32, "warmup": W32,
                    "ms_per_step": r32["ms"] / K32, "batch": wl32.batch, "prompt_len": wl32.prompt_len,
                    "tau": tau, "kv_dtype": wl32.kv_dtype, "gpu_launches": r32["launches"],
                    "context_during_timing": [r32["ctx_begin"], r32["ctx_begin"] + K32 * tau],
                    "roofline": roofline_of(shape, wl32, tau, r32, K32, peak, peak_src),
                    "speedup_vs_tau1": tps32 / tps32_1, "tau1_tokens_per_s": tps32_1, "clocks": clocks32}
            eng32.close()
            del eng32
        del weights
        torch.cuda.empty_cache()

    ms_max, tokens = replicas.aggregate(ms, B * tau * K, device="cuda")
    value = tokens / (ms_max * 1e-3)
    if rank != 0:
        return

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_max / K, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": f"bf16 weights, {wl.kv_dtype} KV cache, fp32 accumulate" if shape.dtype == "bf16" else "f32",
        "data": "synthetic",
        "config": {"workload": wl.name, "shape": wl.shape, "tau": tau, "L_d": L_d, "batch": B,
                   "prompt_len": P, "context_during_timing": [res["ctx_begin"], res["ctx_begin"] + K * tau],
                   "l2": "inputs_exceed_l2 (weights streamed per cycle >> 126 MB)",
                   "parallelism": "replicas" if world > 1 else "single", "device_memory_gb": memory},
        "clocks": clocks,
        "gpu_launches": launches,
        "e2e": {"value": e2e_request, "unit": UNIT,
                "h2d_bytes_per_step": B * P * 4 / max(calls, 1), "d2h_bytes_per_step": B * tau * 4,
                "note": "whole request: prompt upload + prefill + decode with per-cycle token read-back",
                "decode_only_value": e2e_decode,
                "prefill_ms": None if args.no_e2e else e2e_prefill_ms,
                "prefill": None if args.no_e2e else prefill},
        "roofline": roofline_of(shape, wl, tau, res, K, peak, peak_src),
        "speedup_vs_tau1": (value / world / tau1) if tau1 else None,
        "tau1_tokens_per_s": tau1,
        "ms_per_cycle_min_med_max": [min(per_cycle), sorted(per_cycle)[len(per_cycle) // 2], max(per_cycle)],
    }
    if bs32 is not None:
        line["bs32"] = bs32
    if wh is not None:
        steps_cpu = 3
        tps, _, cores = time_oracle(shape, wh, L_d, tau, steps_cpu, 1)
        line["cpu_baseline"] = {"value": tps, "unit": UNIT, "cores": cores, "kind": "oracle",
                                "sample": f"{steps_cpu} decode cycles (tau={tau}) of one sequence after an 8-token "
                                          f"prompt, 1 warm-up cycle, whole model"}
    print(json.dumps(line), flush=True)


def dry_run_replicas(args):
    """The replica protocol of run_native without the GPU work: rendezvous over gloo, barrier on both
    sides of a stand-in for the timed region, max-over-ranks time, summed units, one line from rank 0."""
    from paper_2510_11958_b200 import replicas
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    assert world == args.gpus, f"--gpus {args.gpus} but WORLD_SIZE={world}"
    if world > 1:
        replicas.init_from_env("gloo")
    replicas.barrier()
    ms, units = 10.0 + rank, 100.0
    replicas.barrier()
    ms_max, total = replicas.aggregate(ms, units)
    if rank == 0:
        print(json.dumps({"dry_run": True, "n_gpus": world, "ms_max": ms_max, "units": total}), flush=True)


def spawn_replicas(args):
    """`python bench.py --gpus N` without a launcher: start N replica processes (one per GPU) with
    the rendezvous variables torchrun would set, and pass rank 0's line through."""
    import socket
    import subprocess
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(args.gpus):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(args.gpus),
                   MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen([sys.executable, os.path.abspath(__file__)] + sys.argv[1:], env=env))
    rc = 0
    for p in procs:
        rc = rc or p.wait()
    sys.exit(rc)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="qwen3_4b_b1")
    ap.add_argument("--tau", type=int, default=None)
    ap.add_argument("--kv-dtype", default=None, choices=["f32", "bf16", "f16"], help="KV cache type (default: the workload's)")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="a dmtd_set_option setting of the measured engine, e.g. tcgen05_gemm_stages=4 (repeatable)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-tau1", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-bs32", dest="bs32", action="store_false",
                    help="skip the batch-32 measurement that the default workload's line carries")
    ap.add_argument("--bs32-steps", type=int, default=20)
    ap.add_argument("--dry-run-replicas", action="store_true",
                    help="replica plumbing only (rendezvous, barrier, aggregation) on the gloo backend, no GPU work")
    args = ap.parse_args()
    if args.steps is None:
        # 84 cycles of tau = 3 reproduce the 256-token generation of the headline workload; the
        # CPU reference arm needs seconds per cycle, so its default is shorter
        args.steps = 84 if args.impl == "native" else 10
    args.warmup = max(args.warmup, 3) if args.impl == "native" else args.warmup
    wl = WORKLOADS[args.workload]
    if args.kv_dtype:
        import dataclasses
        wl = dataclasses.replace(wl, kv_dtype=args.kv_dtype)
    args.tau = args.tau or wl.tau
    shape = SHAPES[wl.shape]
    if args.gpus > 1 and "RANK" not in os.environ and args.impl == "native":
        spawn_replicas(args)                # does not return; the reference arm is rank 0 alone
    if args.dry_run_replicas:
        return dry_run_replicas(args)
    if args.impl == "reference":
        run_reference(args, wl, shape)
    else:
        run_native(args, wl, shape)


if __name__ == "__main__":
    main()

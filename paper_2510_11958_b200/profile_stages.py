"""Per-stage time stamps of the persistent pass kernel.

    python -m paper_2510_11958_b200.profile_stages [--workload qwen3_4b_b1] [--kind full|upper]

Builds a profiling variant of the library (-DDMTD_PASS_TIMING, written beside the normal one as
libdmtd_b200_timing.so), runs a few decode cycles of the workload and prints, for the first and
the last block of the grid, how long thread 0 spent in every prologue, projection and grid
barrier of one pass, averaged over the layers.  Times are clock64() ticks converted with
the SM clock the launch itself measured (ticks between kernel entry and exit over the wall clock's
nanoseconds; about 1.86 GHz under this load), or with --ghz.
"""
import argparse
import ctypes as C
import os
import subprocess
import sys

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
LIB = os.path.join(HERE, "libdmtd_b200_timing.so")
SLOTS = 4096
NAMES = ["qkv_pro", "qkv_mma", "qkv_bar", "attn", "-", "attn_bar", "o_pro", "o_mma", "o_bar",
         "gu_pro", "gu_mma", "gu_bar", "dn_pro", "dn_mma", "dn_bar"]


def build_timing_library():
    nvcc = os.environ.get("NVCC", "/usr/local/cuda/bin/nvcc")
    cmd = [nvcc, "-gencode", "arch=compute_100a,code=sm_100a", "-O3", "-lineinfo", "-std=c++17",
           "-DDMTD_PASS_TIMING", "-Xcompiler", "-fPIC", "-shared", "-I", os.path.join(ROOT, "include"),
           os.path.join(HERE, "csrc", "engine.cu"), "-o", LIB] + os.environ.get("DMTD_NVCC_FLAGS", "").split()
    subprocess.run(cmd, check=True)
    return LIB


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="qwen3_4b_b1")
    ap.add_argument("--kind", default="full", choices=["full", "upper"])
    ap.add_argument("--ghz", type=float, default=None, help="SM clock for tick -> us (default: measured in the launch itself)")
    ap.add_argument("--kv", default=None, choices=["bf16", "f16", "f32"], help="KV cache type (default: the workload's)")
    ap.add_argument("--prompt-len", type=int, default=None, help="prompt length (default: the workload's)")
    ap.add_argument("--option", action="append", default=[], metavar="NAME=VALUE",
                    help="a dmtd_set_option setting for the run, e.g. prefetch_chunks=0 (repeatable)")
    ap.add_argument("--build-only", action="store_true")
    args = ap.parse_args()
    build_timing_library()
    if args.build_only:
        return
    sys.path.insert(0, ROOT)
    import torch
    from paper_2510_11958_b200 import binding as bd
    from synthetic import SHAPES, WORKLOADS, make_prompts, make_weights
    bd.library_path = lambda: LIB
    wl = WORKLOADS[args.workload]
    if args.prompt_len:
        import dataclasses
        wl = dataclasses.replace(wl, prompt_len=args.prompt_len)
    shape = SHAPES[wl.shape]
    w = make_weights(shape, seed=wl.weight_seed, device="cuda")
    eng = bd.Dmtd(shape, w, L_d=wl.L_d, tau=wl.tau, max_batch=wl.batch, max_seq=wl.prompt_len + 64,
                  kv_dtype=args.kv or wl.kv_dtype)
    del w
    for kv in args.option:
        name, value = kv.split("=")
        eng.set_option(name, int(value))
    eng.prefill(make_prompts(shape.vocab, wl.batch, wl.prompt_len, seed=wl.prompt_seed).cuda())
    for _ in range(4):
        eng.decode_cycle(wl.tau)                     # ends at a cycle boundary: the next pass is a full one
    if args.kind == "upper":
        eng.decode_cycle(1)
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2)]
    ev[0].record()
    eng.decode_cycle(1)
    ev[1].record()
    torch.cuda.synchronize()
    print(f"{args.workload}, KV {args.kv or wl.kv_dtype}, {args.kind} pass: {ev[0].elapsed_time(ev[1]) * 1e3:.1f} us by CUDA events")
    buf = np.zeros(2 * SLOTS, np.int64)
    eng.dll.dmtd_debug_pass_timing.argtypes = [C.c_void_p, C.c_void_p]
    assert eng.dll.dmtd_debug_pass_timing(eng._ctx, buf.ctypes.data_as(C.c_void_p)) == 0
    n_layers = shape.n_layers if args.kind == "full" else wl.L_d
    if args.ghz is None:
        c0, w0, c1, w1 = (int(v) for v in buf[SLOTS - 4:SLOTS])
        args.ghz = (c1 - c0) / max(w1 - w0, 1)           # clock64 ticks per nanosecond of the wall clock
    for blk, label in ((0, "first block"), (1, "last block")):
        s = buf[blk * SLOTS:(blk + 1) * SLOTS]
        n = 1 + n_layers * 15 + 3
        d = np.diff(s[:n]) / (args.ghz * 1e3)
        per = d[: n_layers * 15].reshape(n_layers, 15)
        print(f"{label}: {(s[n - 1] - s[0]) / (args.ghz * 1e3):.1f} us from first to last stamp")
        rest = per[1:] if n_layers > 1 else per          # the first layer of a pass starts with a cold ring
        print("  us per layer (mean over layers 1..): " +
              " ".join(f"{nm}={rest[:, i].mean():.1f}" for i, nm in enumerate(NAMES) if nm != "-") +
              f" | sum {rest.mean(0).sum():.1f}")
        print("  head: prologue %.1f, projection %.1f, barrier %.1f" % tuple(d[n_layers * 15: n_layers * 15 + 3]))
        if blk == 0:
            a = s[SLOTS - 20:SLOTS - 12]
            print("  inside the last layer's attention stage (entry, rows requested, cached tile fetched, rows landed, "
                  "rows normed, tiles done, partials stored, exit): " + " ".join(f"{v / (args.ghz * 1e3):.2f}" for v in np.diff(a)))
            i_bar = 1 + (n_layers - 1) * 15 + 2                 # stamp after the last layer's QKV barrier; + 1: after its attention stage
            print("  last layer: %.2f us from the QKV barrier's end to the attention stage's first stamp, %.2f us from its last stamp to the stage's end"
                  % ((a[0] - s[i_bar]) / (args.ghz * 1e3), (s[i_bar + 1] - a[7]) / (args.ghz * 1e3)))
            t = s[SLOTS - 12:SLOTS - 5]
            print("  last tile: sync %.2f, new rows placed %.2f, copies landed + sync %.2f, multiplied %.2f" %
                  tuple(v / (args.ghz * 1e3) for v in (t[0] - a[4], t[1] - t[0], t[2] - t[1], a[5] - t[2])))
            if t[6] > t[2]:
                print("  multiplied = scores %.2f, sync %.2f, softmax %.2f, sync %.2f, P V %.2f (fp32 cache only)" %
                      tuple(v / (args.ghz * 1e3) for v in (t[3] - t[2], t[4] - t[3], t[5] - t[4], t[6] - t[5], a[5] - t[6])))
        if blk == 0:
            print("  last layer, the chunks of a warp's share: waited + consumed (us); last figure: the share took")
            for pi, pname in enumerate(("qkv", "o", "gate/up", "down")):
                for wi, wname in enumerate(("warp 0", "warp 7")):
                    c = s[2048 + 64 * pi + 32 * wi: 2048 + 64 * pi + 32 * wi + 32]
                    c = c[c > 0]
                    if len(c) > 2:
                        d = np.diff(c) / (args.ghz * 1e3)
                        print(f"    {pname:8s}{wname}: " + " ".join(f"{d[i]:.2f}+{d[i + 1]:.2f}" for i in range(0, len(d) - 1, 2)) +
                              f" | {(c[-1] - c[0]) / (args.ghz * 1e3):.2f}")
        if blk == 0:
            us = lambda a: " ".join(f"{v / (args.ghz * 1e3):.2f}" for v in np.diff(a))
            print("  inside the last norm prologue (rows and norm weights requested, rows landed, squares summed, "
                  "columns written, block barrier): " + us(s[3072:3078]))
            for pi, pname in enumerate(("qkv", "o", "gate/up", "down", "attention")):
                f = s[3200 + 160 * pi: 3200 + 160 * pi + 160]
                f = f[f > 0].astype(np.float64)
                if len(f):
                    f = (f - f.min()) / 1e3
                    order = np.argsort(f)
                    print(f"  last layer, {pname}: blocks done within {f.max():.2f} us of the first (median {np.median(f):.2f}); "
                          f"last five blocks {[int(v) for v in order[-5:]]} at " + " ".join(f"{v:.2f}" for v in f[order[-5:]]) +
                          f"; by block index, means of 4 groups of 37: " + " ".join(f"{f[i * 37:(i + 1) * 37].mean():.2f}" for i in range(4)))
            print("  inside the last grid barrier (block barrier, arrive + poll, block barrier): " + us(s[3088:3092]))
        c0, w0, c1, w1 = (int(v) for v in s[SLOTS - 4:])
        print(f"  kernel entry to exit: {(w1 - w0) / 1e3:.1f} us by the wall clock, SM clock {(c1 - c0) / max(w1 - w0, 1):.3f} GHz; "
              f"entry to first stamp {(s[0] - c0) / (args.ghz * 1e3):.1f} us, last stamp to exit {(c1 - s[n - 1]) / (args.ghz * 1e3):.1f} us")


if __name__ == "__main__":
    main()

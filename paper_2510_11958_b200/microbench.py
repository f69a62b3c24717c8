"""Single-layer microbenchmark: one decode step of one Qwen3-4B-shaped layer over a grid of batch
sizes and KV lengths, with random hidden states and a random KV cache.

    python -m paper_2510_11958_b200.microbench [--batches 1,8,64,256] [--kv 1024,8192,32768]

For every cell it times (CUDA events, inputs far larger than L2 or an L2 flush between
iterations) the whole layer through dmtd_step_layers and the attention alone through
dmtd_attention_decode, and prints one JSON line with the achieved GB/s of each against the
bytes the step must move: the layer's weights (201.86 MB) once, and K and V of every cached
position of every sequence once.
"""
import argparse
import ctypes as C
import json
import os
import sys

import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2510_11958_b200 import Dmtd, attention_decode  # noqa: E402
from synthetic import SHAPES, make_weights, weight_bytes  # noqa: E402


def fill_kv_random(eng, shape, B, S, seed):
    """N(0, 1) into positions [0, S) of layer 0's cache, one sequence at a time."""
    rt = C.CDLL("libcudart.so")
    kp, vp = eng.kv(0)
    g = torch.Generator(device="cuda").manual_seed(seed)
    per_seq = shape.n_kv_heads * eng.max_seq * shape.head_dim
    for b in range(B):
        for ptr in (kp, vp):
            t = torch.randn(shape.n_kv_heads, eng.max_seq, shape.head_dim, generator=g, device="cuda").to(torch.bfloat16)
            rt.cudaMemcpy(C.c_void_p(ptr + b * per_seq * 2), C.c_void_p(t.data_ptr()), C.c_size_t(per_seq * 2), 3)
    torch.cuda.synchronize()


def time_ms(fn, iters, flush):
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * iters)]
    for i in range(3):
        fn()
    total = 0.0
    for i in range(iters):
        if flush is not None:
            flush.zero_()                       # larger than L2: the next iteration starts cold
        ev[2 * i].record()
        fn()
        ev[2 * i + 1].record()
    torch.cuda.synchronize()
    for i in range(iters):
        total += ev[2 * i].elapsed_time(ev[2 * i + 1])
    return total / iters


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--batches", default="1,8,64,256")
    ap.add_argument("--kv", default="1024,8192,32768")
    ap.add_argument("--iters", type=int, default=10)
    args = ap.parse_args()
    shape = SHAPES["qwen3_4b"].with_(n_layers=1, vocab=1024)      # the layer is what is timed; a small tied head
    w_layer, _ = weight_bytes(shape)
    weights = make_weights(shape, seed=2, device="cuda")
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    peaks = os.path.join(ROOT, "MEASURED_PEAKS.json")
    peak = json.load(open(peaks))["hbm_gbs"] if os.path.exists(peaks) else 6650.0
    for B in [int(x) for x in args.batches.split(",")]:
        for S in [int(x) for x in args.kv.split(",")]:
            eng = Dmtd(shape, weights, L_d=1, tau=1, max_batch=B, max_seq=S + 1, kv_dtype="bf16")
            fill_kv_random(eng, shape, B, S, seed=2)
            g = torch.Generator(device="cuda").manual_seed(3)
            hidden = torch.randn(B, 1, shape.hidden, generator=g, device="cuda")
            h = hidden.clone()

            def layer():
                h.copy_(hidden)
                eng.step_layers(0, 1, h, S)

            kv_bytes = B * S * 2 * shape.n_kv_heads * shape.head_dim * 2
            t_layer = time_ms(layer, args.iters, flush)
            # attention alone on the same cache (position S holds the K, V the layer step appended)
            kp, vp = eng.kv(0)
            q = torch.randn(B, 1, shape.n_q_heads, shape.head_dim, generator=g, device="cuda")
            n = B * shape.n_kv_heads * (S + 1) * shape.head_dim
            k_t = torch.empty(n, dtype=torch.bfloat16, device="cuda")
            v_t = torch.empty(n, dtype=torch.bfloat16, device="cuda")
            rt = C.CDLL("libcudart.so")
            rt.cudaMemcpy(C.c_void_p(k_t.data_ptr()), C.c_void_p(kp), C.c_size_t(n * 2), 3)
            rt.cudaMemcpy(C.c_void_p(v_t.data_ptr()), C.c_void_p(vp), C.c_size_t(n * 2), 3)
            k_t = k_t.view(B, shape.n_kv_heads, S + 1, shape.head_dim)
            v_t = v_t.view(B, shape.n_kv_heads, S + 1, shape.head_dim)
            t_attn = time_ms(lambda: attention_decode(q, k_t, v_t, S), args.iters, flush)
            line = {"bench": "single layer decode step", "shape": "qwen3_4b layer", "batch": B, "kv_len": S,
                    "layer_ms": t_layer, "layer_bytes": w_layer + kv_bytes,
                    "layer_gbs": (w_layer + kv_bytes) / (t_layer * 1e-3) / 1e9,
                    "attention_ms": t_attn, "attention_bytes": kv_bytes,
                    "attention_gbs": kv_bytes / (t_attn * 1e-3) / 1e9,
                    "projections_ms_by_difference": t_layer - t_attn,
                    "projections_gbs_by_difference": w_layer / max(t_layer - t_attn, 1e-6) / 1e6,
                    "projection_kernel": "gemv_bf16 (mma.sync)" if B <= 4 else "gemm_tc05 (tcgen05)",
                    "hbm_peak_gbs": peak, "layer_frac_of_peak": (w_layer + kv_bytes) / (t_layer * 1e-3) / 1e9 / peak,
                    "l2": "flushed between iterations"}
            print(json.dumps(line), flush=True)
            del eng, k_t, v_t
            torch.cuda.empty_cache()


if __name__ == "__main__":
    main()

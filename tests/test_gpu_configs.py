"""Parity at the sizes the five benchmark configurations name, through the launch configurations
`bench.py` times.  The oracle's cost bounds every case; each docstring states the subset taken.

  config 2  Qwen3-4B shape, batch 1, 512-token prompt, tau = 3, L_d = 8: all 36 layers, every pass
            teacher-forced, the first 96 of the 255 decode passes (the oracle needs about 100 s for
            the prefill and half a second per pass on 16 cores).
  config 3  the same layer geometry at batch 32, tau in {1, 2, 3, 4} (32 .. 128 rows in the lower
            layers): 4 layers, short prompts, sequences 0 and 31 through the oracle.
  config 4  batch 8, 16 384-token prompts, bf16 KV cache: one layer at 16 384 cached positions against
            the oracle's layer, and a 2048-token prompt through 4 layers for two cycles.
  config 5  one decoding layer over the grid batch {1, 8, 64, 256} x KV length {1024, 8192, 32768}:
            every cell's output rows against the oracle's layer (sequences 0 and B-1 where B >= 64).
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from synthetic import SHAPES, make_prompts, make_weights

from helpers import LOGIT_ATOL, check_logits, gpu_forced, oracle_forced, to_cuda

pytestmark = pytest.mark.gpu

# Measured on the 36-layer model (readings): a bf16 KV cache alone moves the logits by
# about 0.06 at full depth, which is why the workloads whose logits are held to 2e-2 keep an fp32
# cache.  The bound asserted below is that measurement with head-room, so that a kernel fault in the
# bf16 attention path (errors of order 1) cannot hide behind it.
BF16_KV_FULL_DEPTH_BOUND = 0.12


@pytest.fixture(scope="module")
def dmtd():
    import paper_2510_11958_b200 as pkg
    pkg.load_library()
    return pkg


class _DevView:
    """A raw device pointer as something torch can wrap (no copy)."""

    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr, "data": (int(ptr), False),
                                         "version": 2}


def _kv_views(eng, layer, B, nkv, max_seq, D):
    """K and V of one layer of a bf16-cache context as torch tensors [B, nkv, max_seq, D] (views)."""
    kp, vp = eng.kv(layer)
    out = []
    for p in (kp, vp):
        raw = torch.as_tensor(_DevView(p, (B, nkv, max_seq, D), "<i2"), device="cuda")
        out.append(raw.view(torch.bfloat16))
    return out


def test_config2_full_depth_prompt_512_teacher_forced(dmtd):
    """Config 2 at its own sizes: 36 layers, full vocabulary, 512-token prompt, the persistent pass
    kernel on every decode pass, with the fp16 KV cache the benchmark workload uses and with an fp32
    one.  97 tokens: the prefill's and 96 decode passes (32 whole cycles), logits of every pass
    against the oracle."""
    shape = SHAPES["qwen3_4b"]
    P, n_new, L_d, tau = 512, 97, 8, 3
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, 1, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, n_new, seed=2).numpy()
    ref_logits, ref_am, o = oracle_forced(shape, w, L_d, tau, prompts, forced)
    wc = to_cuda(w)
    del w
    for kv in ("f16", "f32"):
        eng = dmtd.Dmtd(shape, wc, L_d=L_d, tau=tau, max_batch=1, max_seq=P + n_new + 1, kv_dtype=kv)
        l0 = eng.launch_count()
        got_logits, got_am = gpu_forced(eng, prompts, forced)
        err, clear = check_logits(got_logits, ref_logits, got_am, ref_am)
        assert eng.device_state() == o.state()
        print(f"config 2, {n_new - 1} decode passes, {kv} cache: max|dlogit|={err:.2e}, clear-margin steps {clear:.0%}, "
              f"launches {eng.launch_count() - l0}")
        eng.close()


def test_full_depth_bf16_kv_cache_measured_bound(dmtd):
    """The long-context configuration names a bf16 KV cache.  At full depth that choice by itself
    costs more than the 2e-2 logit tolerance; this test measures what it costs (36 layers, full
    vocabulary, both CUDA paths) and holds it to the recorded bound, next to the same run with an
    fp32 cache, which must meet 2e-2."""
    shape = SHAPES["qwen3_4b"]
    P, n_new, L_d, tau = 40, 9, 8, 3
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, 1, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, n_new, seed=2).numpy()
    ref_logits, ref_am, o = oracle_forced(shape, w, L_d, tau, prompts, forced)
    wc = to_cuda(w)
    del w
    seen = {}
    for kv, fused in (("f32", 1), ("bf16", 1), ("bf16", 0), ("f16", 0), ("f16", 1)):
        eng = dmtd.Dmtd(shape, wc, L_d=L_d, tau=tau, max_batch=1, max_seq=P + n_new + 1, kv_dtype=kv)
        eng.set_option("fused_pass", fused)
        got_logits, got_am = gpu_forced(eng, prompts, forced)
        err = float(np.abs(got_logits - ref_logits).max())
        seen[(kv, fused)] = err
        assert eng.device_state() == o.state()
        eng.close()
    print("full depth, max|dlogit|: " + ", ".join(f"{k[0]} cache/{'pass kernel' if k[1] else 'per-step'} {v:.3e}"
                                                    for k, v in seen.items()))
    assert seen[("f32", 1)] <= LOGIT_ATOL
    assert seen[("bf16", 1)] <= BF16_KV_FULL_DEPTH_BOUND
    assert seen[("bf16", 0)] <= BF16_KV_FULL_DEPTH_BOUND
    # an fp16 cache (the batch-1 and batch-32 workloads': half of fp32's bytes, tensor-core attention) meets the tolerance
    assert seen[("f16", 0)] <= LOGIT_ATOL
    assert seen[("f16", 1)] <= LOGIT_ATOL


@pytest.mark.parametrize("tau,kv", [(1, "f16"), (2, "f16"), (3, "f16"), (4, "f16"), (3, "f32")])
def test_config3_batch32_4b_geometry(dmtd, tau, kv):
    """Config 3's layer geometry (hidden 2560, 32/8 heads, intermediate 9728, full vocabulary) at batch
    32: 32 tau rows in the lower layers (32, 64, 96, 128: the tcgen05 GEMM with its k-split, the
    two-blocks-per-SM gate+up case at 96 rows) and 32 in the decoding layers; 4 layers, L_d = 2, the
    fp16 KV cache of the batch-32 workload (and once an fp32 cache).  Sequences 0 and 31 go through the oracle one by one (sequences are independent);
    every pass's logits of those two are compared, and the device counters."""
    shape = SHAPES["qwen3_4b_l4"]
    B, P, L_d = 32, 40, 2
    n_new = 1 + (tau - 1) + 2 * tau                       # cycle 1 and two whole cycles
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, n_new, seed=2).numpy()
    eng = dmtd.Dmtd(shape, to_cuda(w), L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 1, kv_dtype=kv)
    got_logits, got_am = gpu_forced(eng, prompts, forced)
    worst = 0.0
    for b in (0, B - 1):
        ref_logits, ref_am, o = oracle_forced(shape, w, L_d, tau, prompts[b:b + 1], forced[b:b + 1])
        err, _ = check_logits(got_logits[:, b:b + 1], ref_logits, got_am[:, b:b + 1], ref_am)
        worst = max(worst, err)
        assert eng.device_state() == o.state()
    # the same batch with the projections on the mma.sync GEMV: the two GEMM paths agree
    eng2 = dmtd.Dmtd(shape, to_cuda(w), L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 1, kv_dtype=kv)
    eng2.set_option("tcgen05_gemm", 0)
    alt_logits, _ = gpu_forced(eng2, prompts, forced)
    # not bit-equal: a last-bit difference in k or v can flip its rounding in a 16-bit cache
    assert np.abs(alt_logits - got_logits).max() < (2e-3 if kv == "f32" else 5e-3)
    print(f"config 3, tau={tau} ({B * tau} rows), {kv} cache: max|dlogit|={worst:.2e}")


def _random_cell(dmtd, B, S, seed, oracle_rows):
    """One decoding layer of the 4B geometry, random N(0,1) hidden rows and KV cache drawn on the GPU
    (the oracle reads back the sequences it checks).  Returns (max error, scale of the reference)."""
    shape = SHAPES["qwen3_4b"].with_(n_layers=1, vocab=512)
    w = make_weights(shape, seed=2)
    nkv, D = shape.n_kv_heads, shape.head_dim
    eng = dmtd.Dmtd(shape, to_cuda(w), L_d=1, tau=1, max_batch=B, max_seq=S + 1, kv_dtype="bf16")
    g = torch.Generator(device="cuda").manual_seed(seed)
    kd, vd = _kv_views(eng, 0, B, nkv, S + 1, D)
    step = max(1, (1 << 28) // (nkv * (S + 1) * D))              # sequences filled per call, bounded memory
    for b0 in range(0, B, step):
        n = min(step, B - b0)
        for dst in (kd, vd):
            dst[b0:b0 + n] = torch.randn(n, nkv, S + 1, D, generator=g, device="cuda").to(torch.bfloat16)
    hidden = torch.randn(B, 1, shape.hidden, generator=g, device="cuda")
    o = oracle.Oracle(shape, w, L_d=1, tau=1, max_batch=len(oracle_rows), max_seq=S + 1)
    for i, b in enumerate(oracle_rows):
        o.set_kv(0, i, kd[b, :, :S].double().permute(1, 0, 2).cpu().numpy(),
                 vd[b, :, :S].double().permute(1, 0, 2).cpu().numpy())
    ref = o.step_layers(0, 1, hidden[oracle_rows].double().cpu().numpy(), S)
    got = eng.step_layers(0, 1, hidden.clone(), S)
    torch.cuda.synchronize()
    err = np.abs(got[oracle_rows].double().cpu().numpy() - ref).max()
    eng.close()
    return float(err), float(np.abs(ref).max())


@pytest.mark.parametrize("B", [1, 8, 64, 256])
@pytest.mark.parametrize("S", [1024, 8192, 32768])
def test_config5_single_layer_grid(dmtd, B, S):
    """Every cell of the single-layer microbenchmark grid: one decode step of one layer in the 4B
    geometry with a bf16 cache of S random positions per sequence, output rows against the oracle's
    layer on the same values (all sequences where B <= 8, sequences 0 and B-1 otherwise)."""
    rows = list(range(B)) if B <= 8 else [0, B - 1]
    err, scale = _random_cell(dmtd, B, S, seed=100 + B + S, oracle_rows=rows)
    # bf16 cache on the tensor cores: Q, P and the appended K, V are rounded to bf16 (2^-9 relative)
    assert err <= 4e-3 * max(1.0, scale), (err, scale)


def test_config4_layer_cell_at_16k_context(dmtd):
    """Config 4's context length: batch 8, 16 384 cached positions per sequence, bf16 cache; all 8
    sequences of one decode step of one layer against the oracle's layer."""
    err, scale = _random_cell(dmtd, 8, 16384, seed=77, oracle_rows=list(range(8)))
    assert err <= 4e-3 * max(1.0, scale), (err, scale)


def test_config4_prompt_2048_two_cycles_bf16_kv(dmtd):
    """The long-context workload scaled to what the oracle can prefill (2048-token prompt, 4 layers
    of the 4B geometry, batch 2, tau = 3): the prefill in several chunks, cycle 1's two short passes
    and two whole cycles, teacher-forced, logits of every pass.  With the bf16 cache the
    configuration names the logits are held to the bound measured for that cache; the same run with
    an fp32 cache must meet 2e-2, which separates the cache's rounding from a kernel fault."""
    shape = SHAPES["qwen3_4b_l4"]
    B, P, L_d, tau, n_new = 2, 2048, 2, 3, 9
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, n_new, seed=2).numpy()
    ref_logits, ref_am, o = oracle_forced(shape, w, L_d, tau, prompts[:1], forced[:1])
    wc = to_cuda(w)
    seen = {}
    for kv in ("f32", "bf16"):
        eng = dmtd.Dmtd(shape, wc, L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 1, kv_dtype=kv)
        got_logits, got_am = gpu_forced(eng, prompts, forced)
        seen[kv] = np.abs(got_logits[:, :1] - ref_logits).max(axis=(1, 2))
        assert eng.device_state() == o.state()
        eng.close()
    print("config 4 stand-in (P=2048, 4 layers), max|dlogit| per pass: f32 cache "
          + " ".join(f"{e:.1e}" for e in seen["f32"]) + "; bf16 cache " + " ".join(f"{e:.1e}" for e in seen["bf16"]))
    assert seen["f32"].max() <= LOGIT_ATOL
    assert seen["bf16"].max() <= BF16_KV_FULL_DEPTH_BOUND

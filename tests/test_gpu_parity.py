"""Parity of the CUDA library (through its C ABI) with the CPU oracle, element by element."""
import numpy as np
import pytest
import torch

from synthetic import SHAPES, make_prompts, make_weights

from helpers import (LOGIT_ATOL, check_logits, gpu_forced, oracle_forced, oracle_greedy, to_cuda)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dmtd():
    import paper_2510_11958_b200 as pkg
    pkg.load_library()
    return pkg


def _engine(dmtd, shape, wc, L_d, tau, max_batch, max_seq, **kw):
    return dmtd.Dmtd(shape, wc, L_d=L_d, tau=tau, max_batch=max_batch, max_seq=max_seq, **kw)


CASES = [
    # name, shape, dtype, L_d, tau, B, P, n_new
    ("tiny_f32_tau3", "tiny", "f32", 2, 3, 1, 32, 24),
    ("tiny_f32_tau1", "tiny", "f32", 2, 1, 1, 32, 24),
    ("tiny_bf16_tau3", "tiny", "bf16", 2, 3, 1, 32, 24),
    ("tiny_bf16_b3_tau4", "tiny", "bf16", 1, 4, 3, 7, 14),
    ("mid_bf16_tau3", "mid", "bf16", 2, 3, 2, 37, 13),
    ("mid_bf16_tau2_b5", "mid", "bf16", 4, 2, 5, 9, 8),
    ("mid_bf16_Ld_all", "mid", "bf16", 6, 3, 1, 11, 7),
]


@pytest.mark.parametrize("name,shape_name,dtype,L_d,tau,B,P,n_new", CASES, ids=[c[0] for c in CASES])
def test_teacher_forced_logits_and_state(dmtd, name, shape_name, dtype, L_d, tau, B, P, n_new):
    shape = SHAPES[shape_name].with_(dtype=dtype)
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    # teacher sequence: what the oracle itself generates greedily
    toks, _, _, _ = oracle_greedy(shape, w, L_d, tau, prompts, n_new)
    ref_logits, ref_am, o = oracle_forced(shape, w, L_d, tau, prompts, toks)
    eng = _engine(dmtd, shape, to_cuda(w), L_d, tau, B, P + n_new + 1)
    got_logits, got_am = gpu_forced(eng, prompts, toks)
    err, clear = check_logits(got_logits, ref_logits, got_am, ref_am)
    assert eng.state() == o.state()
    assert eng.device_state() == o.state()
    print(f"{name}: max|dlogit|={err:.2e}, clear-margin steps {clear:.0%}")


@pytest.mark.parametrize("graph", [0, 1])
@pytest.mark.parametrize("shape_name,dtype,L_d,tau,B,P,n_new", [("tiny", "f32", 2, 3, 1, 32, 24),
                                                               ("mid", "bf16", 2, 3, 2, 20, 17),
                                                               ("tiny", "bf16", 2, 1, 2, 5, 6)])
def test_free_running_greedy(dmtd, graph, shape_name, dtype, L_d, tau, B, P, n_new):
    """Greedy generation call by call: token counts, state after every call (bit-exact), and the
    tokens themselves up to the first step where the oracle's margin is not clear."""
    shape = SHAPES[shape_name].with_(dtype=dtype)
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    toks, logits, states, _ = oracle_greedy(shape, w, L_d, tau, prompts, n_new)
    eng = _engine(dmtd, shape, to_cuda(w), L_d, tau, B, P + n_new + 1)
    eng.set_option("cuda_graph", graph)
    tok, _ = eng.prefill(torch.from_numpy(prompts).cuda())
    got = [tok.cpu().numpy()]
    assert eng.state() == states[0]
    k = 1
    while len(got) < n_new:
        rc, n, out = eng.decode_cycle(n_new - len(got))
        out = out.cpu().numpy()
        got += [out[:, i] for i in range(n)]
        assert eng.state() == states[k]
        assert eng.device_state() == states[k]
        k += 1
    got = np.stack(got, 1)
    srt = np.sort(logits, -1)
    clear = (srt[..., -1] - srt[..., -2] > 5e-2).T            # [B, n]
    for b in range(B):
        upto = n_new if clear[b].all() else int(np.argmin(clear[b]))
        assert (got[b, :upto] == toks[b, :upto]).all()


def test_graph_replay_matches_plain_launches(dmtd):
    shape = SHAPES["mid"]
    w = to_cuda(make_weights(shape, seed=0))
    prompts = torch.from_numpy(make_prompts(shape.vocab, 2, 16, seed=1).numpy()).cuda()
    outs = []
    for graph in (0, 1):
        eng = _engine(dmtd, shape, w, 2, 3, 2, 64)
        eng.set_option("cuda_graph", graph)
        eng.prefill(prompts)
        toks = []
        for _ in range(6):
            rc, n, out = eng.decode_cycle(3)
            toks.append(out[:, :n].clone())
        outs.append(torch.cat(toks, 1).cpu())
        assert eng.launch_count() > 0
    assert (outs[0] == outs[1]).all()


def test_qk_norm_rope_inside_attention_matches_separate_kernel(dmtd):
    """Step a3 (Section 3.1's QK-norm, RoPE, KV append) run inside the tensor-core attention kernel and as a
    launch of its own: the same generated tokens on the per-step path (5 sequences: more rows than the pass kernel takes)."""
    shape = SHAPES["mid"]
    w = to_cuda(make_weights(shape, seed=0))
    prompts = torch.from_numpy(make_prompts(shape.vocab, 5, 21, seed=1).numpy()).cuda()
    outs, launches = [], []
    for fused in (0, 1):
        eng = _engine(dmtd, shape, w, 2, 3, 5, 64)
        eng.set_option("fused_qk_rope", fused)
        eng.set_option("cuda_graph", 0)
        eng.prefill(prompts)
        before = eng.launch_count()
        toks = []
        for _ in range(4):
            rc, n, out = eng.decode_cycle(3)
            toks.append(out[:, :n].clone())
        outs.append(torch.cat(toks, 1).cpu())
        launches.append(eng.launch_count() - before)
    assert (outs[0] == outs[1]).all()
    assert launches[1] < launches[0]                   # one launch less per layer and pass


def test_prefill_longer_than_one_chunk(dmtd):
    """A prompt that does not fit the workspace in one go is fed in causal chunks."""
    shape = SHAPES["tiny"].with_(dtype="bf16")
    w = make_weights(shape, seed=0)
    P = 300                                   # workspace holds 256 rows
    prompts = make_prompts(shape.vocab, 1, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, 4, seed=2).numpy()
    ref_logits, ref_am, o = oracle_forced(shape, w, 2, 3, prompts, forced)
    eng = _engine(dmtd, shape, to_cuda(w), 2, 3, 1, P + 8)
    got_logits, got_am = gpu_forced(eng, prompts, forced)
    check_logits(got_logits, ref_logits, got_am, ref_am)
    assert eng.device_state() == o.state()


@pytest.mark.parametrize("shape_name,dtype,B,R,pos0", [("tiny", "f32", 2, 3, 5), ("mid", "bf16", 3, 3, 17),
                                                      ("mid", "bf16", 1, 1, 40), ("mid", "bf16", 2, 19, 0)])
def test_step_layers_hidden_and_kv(dmtd, shape_name, dtype, B, R, pos0):
    """dmtd_step_layers against the oracle's: output rows and the K/V they append."""
    import oracle
    shape = SHAPES[shape_name].with_(dtype=dtype)
    w = make_weights(shape, seed=3, norm_jitter=0.1)
    L = shape.n_layers
    g = torch.Generator().manual_seed(5)
    max_seq = pos0 + R + 2
    o = oracle.Oracle(shape, w, L_d=1, tau=1, max_batch=B, max_seq=max_seq)
    eng = _engine(dmtd, shape, to_cuda(w), 1, 1, B, max_seq)
    # history: run pos0 earlier rows through both so the caches hold the same past
    if pos0:
        h0 = torch.randn(B, pos0, shape.hidden, generator=g) * 0.5
        o.step_layers(0, L, h0.double().numpy(), 0)
        eng.step_layers(0, L, h0.cuda().contiguous(), 0)
    h = torch.randn(B, R, shape.hidden, generator=g) * 0.5
    ref = o.step_layers(1, L, h.double().numpy(), pos0) if L > 2 else o.step_layers(0, L, h.double().numpy(), pos0)
    l0 = 1 if L > 2 else 0
    got = eng.step_layers(l0, L, h.cuda().contiguous(), pos0)
    torch.cuda.synchronize()
    scale = np.abs(ref).max()
    # bf16 cache: K, V and (tensor-core attention) Q and P are rounded to bf16, 2^-9 relative each;
    # fp32 cache: hi+lo operands, fp32 accuracy
    rel = 1e-4 if dtype == "f32" else 4e-3
    assert np.abs(got.double().cpu().numpy() - ref).max() <= rel * max(1.0, scale)
    # appended K/V of the last layer
    import ctypes
    kp, vp = eng.kv(L - 1)
    kvdt = torch.float32 if dtype == "f32" else torch.bfloat16
    n = B * shape.n_kv_heads * max_seq * shape.head_dim
    for ptr, which in ((kp, 0), (vp, 1)):
        buf = torch.empty(n, dtype=kvdt, device="cuda")
        ctypes.CDLL("libcudart.so").cudaMemcpy(ctypes.c_void_p(buf.data_ptr()), ctypes.c_void_p(ptr),
                                               ctypes.c_size_t(n * buf.element_size()), 3)
        dev = buf.view(B, shape.n_kv_heads, max_seq, shape.head_dim).double().cpu().numpy()
        for b in range(B):
            refkv = o.kv_cache(L - 1, b, pos0 + R)[which]            # [pos, nkv, d]
            gotkv = dev[b].transpose(1, 0, 2)[: pos0 + R]
            tol = 1e-5 if dtype == "f32" else 2.0 ** -8 * max(1.0, np.abs(refkv).max())
            assert np.abs(gotkv - refkv).max() <= tol


def test_batch_rows_are_independent(dmtd):
    shape = SHAPES["mid"]
    w = to_cuda(make_weights(shape, seed=0))
    prompts = make_prompts(shape.vocab, 4, 12, seed=1)
    forced = make_prompts(shape.vocab, 4, 9, seed=2)
    eng = _engine(dmtd, shape, w, 2, 3, 4, 32)
    full, _ = gpu_forced(eng, prompts.numpy(), forced.numpy())
    for b in (0, 3):
        e1 = _engine(dmtd, shape, w, 2, 3, 1, 32)
        one, _ = gpu_forced(e1, prompts[b:b + 1].numpy(), forced[b:b + 1].numpy())
        # not bit-equal: the fp32 reduction order differs with the batch size, and a last-bit
        # change in k or v can flip its bf16 rounding in the cache; mixing up sequences would
        # show as O(0.1)
        assert np.abs(one[:, 0] - full[:, b]).max() < 5e-3


def test_literal_sum_option(dmtd):
    """The literal reading of Eq. 4 (embedding added to the lower-stack output)."""
    shape = SHAPES["tiny"]
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, 1, 9, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, 8, seed=2).numpy()
    ref_logits, ref_am, _ = oracle_forced(shape, w, 2, 3, prompts, forced, literal_sum=True)
    eng = _engine(dmtd, shape, to_cuda(w), 2, 3, 1, 32)
    eng.set_option("literal_sum", 1)
    got_logits, got_am = gpu_forced(eng, prompts, forced)
    check_logits(got_logits, ref_logits, got_am, ref_am)


def test_reset_and_set_tau(dmtd):
    shape = SHAPES["tiny"]
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, 1, 6, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, 7, seed=2).numpy()
    eng = _engine(dmtd, shape, to_cuda(w), 2, 3, 1, 32)
    gpu_forced(eng, prompts, forced)
    eng.reset()
    eng.set_tau(2)
    ref_logits, ref_am, o = oracle_forced(shape, w, 2, 2, prompts, forced)
    got_logits, got_am = gpu_forced(eng, prompts, forced)
    check_logits(got_logits, ref_logits, got_am, ref_am)
    assert eng.device_state() == o.state()


def test_errors(dmtd):
    shape = SHAPES["tiny"]
    w = to_cuda(make_weights(shape, seed=0))
    S = __import__("paper_2510_11958_b200.binding", fromlist=["STATUS"]).STATUS
    with pytest.raises(dmtd.DmtdError) as e:
        _engine(dmtd, shape, w, 5, 3, 1, 32)
    assert e.value.status == S["SHAPE"]
    with pytest.raises(dmtd.DmtdError) as e:
        _engine(dmtd, shape, w, 2, 0, 1, 32)
    assert e.value.status == S["SHAPE"]
    eng = _engine(dmtd, shape, w, 2, 3, 1, 8)
    with pytest.raises(dmtd.DmtdError) as e:
        eng.decode_cycle(3)
    assert e.value.status == S["STATE"]
    prompts = torch.from_numpy(make_prompts(shape.vocab, 1, 5, seed=1).numpy()).cuda()
    with pytest.raises(dmtd.DmtdError) as e:
        eng.prefill(torch.cat([prompts, prompts], 0))
    assert e.value.status == S["CAPACITY"]
    eng.prefill(prompts)
    with pytest.raises(dmtd.DmtdError) as e:
        eng.prefill(prompts)
    assert e.value.status == S["STATE"]
    rc, n, _ = eng.decode_cycle(3)
    assert rc == 0 and n == 2
    rc, n, _ = eng.decode_cycle(3, allow_capacity=True)     # position 8 does not fit max_seq = 8
    assert rc == S["CAPACITY"] and n == 0
    assert eng.device_state() == eng.state()


@pytest.mark.parametrize("kvdt,B,R,nq,nkv,D,pos0,max_seq", [
    ("bf16", 1, 1, 32, 8, 128, 700, 1024),       # one decode row, several key slices, ragged last slice
    ("bf16", 2, 3, 8, 2, 128, 37, 64),           # a refill chunk: causal among the 3 new rows
    ("f32", 3, 4, 4, 2, 64, 0, 8),               # no history at all
    ("bf16", 1, 5, 16, 1, 128, 2300, 2400),      # 16 query heads per KV head, rows split in blocks, long slices
    ("f32", 2, 3, 8, 2, 128, 300, 512),          # fp32 cache: the FMA kernel
    ("f32", 1, 1, 32, 8, 128, 3000, 3072),
    ("f32", 40, 1, 8, 2, 128, 1500, 1536),       # a batch large enough for long slices: 4 tiles per block, ragged
    ("f32", 24, 3, 8, 2, 128, 1000, 1024),       # the same with a refill chunk (12 query rows per tile)
    ("bf16", 40, 1, 8, 2, 128, 1500, 1536),      # several double-buffered tiles per block
    ("f16", 1, 1, 32, 8, 128, 700, 1024),        # fp16 cache: the tensor-core kernel with fp16 operands
    ("f16", 24, 3, 8, 2, 128, 1000, 1024),
    ("f16", 2, 3, 4, 2, 64, 100, 128),           # head_dim 64: the one-warp-per-key-group kernel
])
def test_attention_decode_matches_oracle(dmtd, oracle_lib, kvdt, B, R, nq, nkv, D, pos0, max_seq):
    """dmtd_attention_decode against the oracle's attention on the same (rounded) K and V."""
    g = torch.Generator().manual_seed(11)
    dt = {"f32": torch.float32, "bf16": torch.bfloat16, "f16": torch.float16}[kvdt]
    q = torch.randn(B, R, nq, D, generator=g)
    k = torch.randn(B, nkv, max_seq, D, generator=g).to(dt)
    v = torch.randn(B, nkv, max_seq, D, generator=g).to(dt)
    got = dmtd.attention_decode(q.cuda(), k.cuda(), v.cuda(), pos0)
    torch.cuda.synchronize()
    n = pos0 + R
    for b in range(B):
        ref = oracle_lib.attention(q[b].double().numpy(), k[b, :, :n].double().permute(1, 0, 2).numpy(),
                                   v[b, :, :n].double().permute(1, 0, 2).numpy(), pos0)
        # head_dim 128 with a bf16 cache runs on the tensor cores: Q and P are rounded to bf16 as well
        # (2^-9 relative each); with an fp32 cache the arithmetic is plain fp32
        # ... and with an fp16 cache to fp16 (2^-12 relative each)
        tol = 5e-3 if (kvdt == "bf16" and D == 128) else 6e-4 if (kvdt == "f16" and D == 128) else 2e-5
        assert np.abs(got[b].double().cpu().numpy() - ref).max() <= tol * max(1.0, np.abs(ref).max())


FUSED_CASES = [
    # name, L_d, tau, B, P, n_new, kv cache type
    ("b1_tau3", 2, 3, 1, 37, 13, "bf16"),
    ("b1_tau4_long_prompt", 2, 4, 1, 300, 9, "bf16"),     # several key slices per kv head
    ("b2_tau2", 4, 2, 2, 9, 8, "bf16"),
    ("b4_tau1", 2, 1, 4, 12, 5, "bf16"),
    ("b1_tau3_all_layers_decode", 6, 3, 1, 11, 7, "bf16"),
    ("b1_tau3_f32kv", 2, 3, 1, 37, 13, "f32"),
    ("b1_tau4_long_prompt_f32kv", 2, 4, 1, 1300, 9, "f32"),    # two key tiles per slice
    ("b1_tau3_long_prompt_bf16kv", 2, 3, 1, 1300, 7, "bf16"),
    ("b2_tau2_f32kv", 4, 2, 2, 9, 8, "f32"),
    ("b1_tau3_f16kv", 2, 3, 1, 37, 13, "f16"),
    ("b1_tau4_long_prompt_f16kv", 2, 4, 1, 1300, 9, "f16"),
]


@pytest.mark.parametrize("name,L_d,tau,B,P,n_new,kv", FUSED_CASES, ids=[c[0] for c in FUSED_CASES])
def test_fused_pass_kernel_teacher_forced(dmtd, name, L_d, tau, B, P, n_new, kv):
    """The one-kernel-per-pass path (at most 4 rows per pass) against the oracle, and against the
    per-step kernels on the same inputs."""
    shape = SHAPES["mid"]
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    toks, _, _, _ = oracle_greedy(shape, w, L_d, tau, prompts, n_new)
    ref_logits, ref_am, o = oracle_forced(shape, w, L_d, tau, prompts, toks)
    wc = to_cuda(w)
    res = {}
    for fused in (1, 0):
        eng = _engine(dmtd, shape, wc, L_d, tau, B, P + n_new + 1, kv_dtype=kv)
        eng.set_option("fused_pass", fused)
        l0 = eng.launch_count()
        got_logits, got_am = gpu_forced(eng, prompts, toks)
        res[fused] = (got_logits, eng.launch_count() - l0)
        err, _ = check_logits(got_logits, ref_logits, got_am, ref_am)
        if kv == "f32":
            assert err < 1e-3                  # nothing is rounded to bf16 but the weights
        assert eng.state() == o.state()
        assert eng.device_state() == o.state()
    # the fused path really ran: one launch per decode pass instead of dozens
    assert res[1][1] < res[0][1]
    assert np.abs(res[1][0] - res[0][0]).max() < 5e-3


def test_fused_pass_kernel_free_running(dmtd):
    shape = SHAPES["mid"]
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    B, P, n_new, L_d, tau = 1, 33, 19, 2, 3
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    toks, logits, states, _ = oracle_greedy(shape, w, L_d, tau, prompts, n_new)
    eng = _engine(dmtd, shape, to_cuda(w), L_d, tau, B, P + n_new + 1)
    tok, _ = eng.prefill(torch.from_numpy(prompts).cuda())
    got = [tok.cpu().numpy()]
    k = 1
    while len(got) < n_new:
        rc, n, out = eng.decode_cycle(n_new - len(got))
        out = out.cpu().numpy()
        got += [out[:, i] for i in range(n)]
        assert eng.device_state() == states[k]
        k += 1
    got = np.stack(got, 1)
    srt = np.sort(logits, -1)
    clear = (srt[..., -1] - srt[..., -2] > 5e-2).T
    for b in range(B):
        upto = n_new if clear[b].all() else int(np.argmin(clear[b]))
        assert (got[b, :upto] == toks[b, :upto]).all()


@pytest.mark.parametrize("B,tau,P,n_new", [(12, 3, 23, 8), (40, 1, 9, 3), (32, 3, 9, 9), (32, 4, 9, 9)])      # 36, 40, 96 and 128 rows per pass
def test_tcgen05_projections_many_rows(dmtd, B, tau, P, n_new):
    """Passes of more than 4 rows run their projections on the tcgen05 GEMM (prefill chunks
    included): against the oracle, and against the mma.sync GEMV on the same inputs.  96 rows is the
    lower-layer row count of batch 32 at tau = 3 (192 accumulator columns in 256 of tensor memory)."""
    shape = SHAPES["mid"].with_(intermediate=1856)          # every K a multiple of the 64-wide k block
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    toks, _, _, _ = oracle_greedy(shape, w, 2, tau, prompts, n_new)
    ref_logits, ref_am, o = oracle_forced(shape, w, 2, tau, prompts, toks)
    wc = to_cuda(w)
    res = {}
    for tc in (1, 0):
        eng = _engine(dmtd, shape, wc, 2, tau, B, P + n_new + 1, kv_dtype="f32")
        eng.set_option("tcgen05_gemm", tc)
        got_logits, got_am = gpu_forced(eng, prompts, toks)
        err, _ = check_logits(got_logits, ref_logits, got_am, ref_am)
        assert err < 1e-3
        assert eng.device_state() == o.state()
        res[tc] = got_logits
    assert np.abs(res[1] - res[0]).max() < 1e-3


@pytest.mark.parametrize("B,S", [(8, 2048), (64, 300), (1, 4100)])
def test_single_layer_cell_random_hidden_and_kv(dmtd, oracle_lib, B, S):
    """A cell of the single-layer microbenchmark (4B layer geometry, random N(0,1) hidden states and
    KV cache, one decode step) against the oracle's layer on the same values."""
    import ctypes
    import oracle
    shape = SHAPES["qwen3_4b"].with_(n_layers=1, vocab=512)
    w = make_weights(shape, seed=2)
    g = torch.Generator().manual_seed(7)
    k = torch.randn(B, shape.n_kv_heads, S, shape.head_dim, generator=g).to(torch.bfloat16)
    v = torch.randn(B, shape.n_kv_heads, S, shape.head_dim, generator=g).to(torch.bfloat16)
    hidden = torch.randn(B, 1, shape.hidden, generator=g)
    o = oracle.Oracle(shape, w, L_d=1, tau=1, max_batch=B, max_seq=S + 1)
    for b in range(B):
        o.set_kv(0, b, k[b].double().permute(1, 0, 2).numpy(), v[b].double().permute(1, 0, 2).numpy())
    ref = o.step_layers(0, 1, hidden.double().numpy(), S)
    eng = _engine(dmtd, shape, to_cuda(w), 1, 1, B, S + 1, kv_dtype="bf16")
    kp, vp = eng.kv(0)
    rt = ctypes.CDLL("libcudart.so")
    per_seq = shape.n_kv_heads * (S + 1) * shape.head_dim
    for ptr, src in ((kp, k), (vp, v)):
        full = torch.zeros(B, shape.n_kv_heads, S + 1, shape.head_dim, dtype=torch.bfloat16)
        full[:, :, :S] = src
        dev = full.cuda()
        rt.cudaMemcpy(ctypes.c_void_p(ptr), ctypes.c_void_p(dev.data_ptr()), ctypes.c_size_t(B * per_seq * 2), 3)
    got = eng.step_layers(0, 1, hidden.cuda().contiguous(), S)
    torch.cuda.synchronize()
    scale = np.abs(ref).max()
    # bf16 cache on the tensor cores: Q, P and the appended K, V rounded to bf16 (2^-9 relative)
    assert np.abs(got.double().cpu().numpy() - ref).max() <= 4e-3 * max(1.0, scale)


def test_device_error_word_reaches_the_synchronising_calls(dmtd):
    """Host-made failures only (no GPU wait is made to run out): a token id outside the vocabulary
    (clamped on the device, reported as INVALID_ARG), and the error word written from the host as a
    device-side wait that gave up would write it (reported as TIMEOUT).  The failure is sticky until
    dmtd_reset, after which the context works as before."""
    from paper_2510_11958_b200.binding import STATUS
    shape = SHAPES["tiny"]
    w = make_weights(shape, seed=0)
    eng = _engine(dmtd, shape, to_cuda(w), 2, 3, 1, 32)
    good = make_prompts(shape.vocab, 1, 6, seed=1)
    bad = good.clone()
    bad[0, 2] = shape.vocab + 7
    with pytest.raises(dmtd.DmtdError) as e:
        eng.prefill_host(bad)
    assert e.value.status == STATUS["INVALID_ARG"]
    out_host = torch.zeros(1, 3, dtype=torch.int32)
    with pytest.raises(dmtd.DmtdError) as e:
        eng.decode_cycle_host(3, out_host)
    assert e.value.status == STATUS["INVALID_ARG"]
    eng.reset()
    first = eng.prefill_host(good)
    assert eng.decode_cycle_host(3, out_host) == 2
    want = out_host.clone()
    # a wait that gave up, as the host would see it
    for word, status in ((3, "TIMEOUT"), (2, "TIMEOUT"), (4, "TIMEOUT"), (1, "INVALID_ARG")):
        eng.debug_set_error_word(word)
        with pytest.raises(dmtd.DmtdError) as e:
            eng.decode_cycle_host(3, out_host)
        assert e.value.status == STATUS[status]
        with pytest.raises(dmtd.DmtdError) as e:
            eng.decode_cycle(3)
        assert e.value.status == STATUS[status]
        with pytest.raises(dmtd.DmtdError) as e:
            eng.device_state()
        assert e.value.status == STATUS[status]
        eng.reset()
        assert (eng.prefill_host(good) == first).all()
        assert eng.decode_cycle_host(3, out_host) == 2
        assert (out_host[:, :2] == want[:, :2]).all()
        assert eng.device_state() == eng.state()


def test_set_tau_at_a_cycle_boundary_in_mid_generation(dmtd):
    """Section 3.7 runs a model trained with one cycle length at others: the cycle length changes
    between cycles of one generation (3 -> 2 -> 4), teacher-forced, against the oracle doing the
    same; both refuse a change in mid-cycle."""
    import oracle
    from paper_2510_11958_b200.binding import STATUS
    shape = SHAPES["mid"]
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    B, P = 2, 11
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, 16, seed=2).numpy()
    plan = [(3, 3), (2, 4), (4, 8)]                  # (cycle length, forced tokens run with it), whole cycles each
    for fused in (1, 0):
        o = oracle.Oracle(shape, w, L_d=2, tau=3, max_batch=B, max_seq=P + 20)
        eng = _engine(dmtd, shape, to_cuda(w), 2, 3, B, P + 20, kv_dtype="f32")
        eng.set_option("fused_pass", fused)
        p = torch.from_numpy(prompts).cuda()
        f = torch.from_numpy(forced).cuda()
        _, lg = eng.prefill(p, forced_first=f[:, 0].contiguous(), want_logits=True)
        _, rl = o.prefill(prompts, forced_first=forced[:, 0])
        assert np.abs(lg.double().cpu().numpy() - rl).max() <= LOGIT_ATOL
        with pytest.raises(dmtd.DmtdError) as e:
            eng.set_tau(2)                           # slot 1: mid-cycle
        assert e.value.status == STATUS["STATE"]
        assert o.set_tau(2) != 0
        at = 1
        for i, (tau, n) in enumerate(plan):
            if i > 0:
                eng.set_tau(tau)
                assert o.set_tau(tau) == 0
            n_run = n - 1 if i == 0 else n            # the prefill was pass 1 of the first cycle
            got, gam = eng.decode_forced(f[:, at:at + n_run].contiguous())
            ref, ram = o.decode_forced(np.ascontiguousarray(forced[:, at:at + n_run]))
            at += n_run
            err, _ = check_logits(got.double().cpu().numpy(), ref, gam.cpu().numpy(), ram)
            assert err < 1e-3
            assert eng.state()["slot"] == 0
            assert eng.device_state() == o.state()


def test_memory_info_and_single_weight_copy(dmtd, monkeypatch):
    """The context reports what it holds; with DMTD_WEIGHT_COPIES=1 the tcgen05 block copy of the
    weights is not built and the projections of every row count run on the atom stream."""
    shape = SHAPES["mid"].with_(intermediate=1856)
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    B, P, n_new = 6, 9, 7
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, n_new, seed=2).numpy()
    ref_logits, ref_am, o = oracle_forced(shape, w, 2, 3, prompts, forced)
    wc = to_cuda(w)
    seen = {}
    for copies in ("2", "1"):
        monkeypatch.setenv("DMTD_WEIGHT_COPIES", copies)
        eng = _engine(dmtd, shape, wc, 2, 3, B, P + n_new + 1, kv_dtype="f32")
        m = eng.memory_info()
        seen[copies] = m
        n_params = shape.n_layers * (shape.params_per_layer - 2 * shape.hidden - 2 * shape.head_dim) + shape.vocab * shape.hidden
        assert m["weight_stream_bytes"] >= 2 * n_params          # bf16, padded to whole tiles
        assert m["kv_cache_bytes"] == 2 * shape.n_layers * B * shape.n_kv_heads * (P + n_new + 1) * shape.head_dim * 4
        got_logits, got_am = gpu_forced(eng, prompts, forced)
        check_logits(got_logits, ref_logits, got_am, ref_am)
    assert seen["2"]["weight_block_bytes"] >= 2 * n_params and seen["1"]["weight_block_bytes"] == 0

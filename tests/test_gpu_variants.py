"""Parity of the variants beside the default greedy schedule: the ExDy layer allocation (Section 2.1,
the paragraph after Eq. 4; Section 3.3) and the masked parallel forward of Eq. 1-5 as one scoring
pass, and sampling inside the fused pick, all through the C ABI against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
from synthetic import SHAPES, make_prompts, make_weights

from helpers import check_logits, gpu_forced, to_cuda

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dmtd():
    import paper_2510_11958_b200 as pkg
    pkg.load_library()
    return pkg


def _oracle_forced(shape, w, L_e, L_d, tau, prompts, forced, literal=False):
    B, P = prompts.shape
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_batch=B, max_seq=P + forced.shape[1] + 1,
                      literal_sum=literal, L_e=L_e)
    tok, lg = o.prefill(prompts, forced_first=forced[:, 0])
    l, am = o.decode_forced(np.ascontiguousarray(forced[:, 1:]))
    return np.concatenate([lg[None], l], 0), np.concatenate([tok[None], am], 0), o


EXDY_CASES = [
    # shape, dtype, L_e, L_d, tau, B, P, n_new, literal
    ("tiny", "f32", 1, 1, 3, 1, 9, 11, False),
    ("tiny", "f32", 1, 2, 2, 2, 5, 8, True),
    ("mid", "bf16", 2, 2, 3, 2, 21, 10, False),
    ("mid", "bf16", 1, 3, 4, 1, 13, 13, False),
    ("mid", "bf16", 3, 3, 3, 3, 7, 7, False),          # no thinking layers left: every pass is full depth
    ("mid", "bf16", 2, 2, 1, 2, 6, 5, False),          # tau = 1
]


@pytest.mark.parametrize("shape_name,dtype,L_e,L_d,tau,B,P,n_new,literal", EXDY_CASES)
def test_exdy_teacher_forced(dmtd, shape_name, dtype, L_e, L_d, tau, B, P, n_new, literal):
    """Encoding layers reused by the short passes: per-pass logits, the model's own choices and the
    schedule counters against the oracle, with graph replay on and off."""
    shape = SHAPES[shape_name].with_(dtype=dtype)
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, n_new, seed=2).numpy()
    ref_logits, ref_am, o = _oracle_forced(shape, w, L_e, L_d, tau, prompts, forced, literal)
    eng = dmtd.Dmtd(shape, to_cuda(w), L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 1, kv_dtype="f32")
    eng.set_option("encoding_layers", L_e)
    eng.set_option("literal_sum", int(literal))
    got_logits, got_am = gpu_forced(eng, prompts, forced)
    err, _ = check_logits(got_logits, ref_logits, got_am, ref_am)
    assert err < 1e-3
    assert eng.state() == o.state()
    assert eng.device_state() == o.state()


def test_exdy_free_running_graph_replay(dmtd):
    """Greedy generation with encoding layers reused: the captured graphs (one per kind of pass)
    give the tokens of plain launches, and the counters follow the oracle's."""
    shape = SHAPES["mid"]
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    B, P, L_e, L_d, tau, n_cycles = 2, 14, 2, 2, 3, 5
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_batch=B, max_seq=P + 3 * n_cycles + 4, L_e=L_e)
    o.prefill(prompts, want_logits=False)
    states = [o.state()]
    for _ in range(n_cycles):
        o.decode_cycle(tau, want_logits=False)
        states.append(o.state())
    outs = []
    for graph in (0, 1):
        eng = dmtd.Dmtd(shape, to_cuda(w), L_d=L_d, tau=tau, max_batch=B, max_seq=P + 3 * n_cycles + 4, kv_dtype="f32")
        eng.set_option("encoding_layers", L_e)
        eng.set_option("cuda_graph", graph)
        eng.prefill(torch.from_numpy(prompts).cuda())
        toks = []
        for k in range(n_cycles):
            rc, n, out = eng.decode_cycle(tau)
            toks.append(out[:, :n].clone())
            assert eng.device_state() == states[k + 1]
        outs.append(torch.cat(toks, 1).cpu())
    assert (outs[0] == outs[1]).all()


def test_exdy_option_errors(dmtd):
    from paper_2510_11958_b200.binding import STATUS
    shape = SHAPES["tiny"]
    eng = dmtd.Dmtd(shape, to_cuda(make_weights(shape, seed=0)), L_d=2, tau=3, max_batch=1, max_seq=32)
    with pytest.raises(dmtd.DmtdError) as e:
        eng.set_option("encoding_layers", 3)              # 3 + 2 > 4 layers
    assert e.value.status == STATUS["SHAPE"]
    eng.set_option("encoding_layers", 1)
    eng.prefill(torch.from_numpy(make_prompts(shape.vocab, 1, 5, seed=1).numpy()).cuda())
    with pytest.raises(dmtd.DmtdError) as e:
        eng.set_option("encoding_layers", 0)              # a property of the whole generation
    assert e.value.status == STATUS["STATE"]


MASKED_CASES = [
    # shape, dtype, L_e, L_d, tau, B, P, n, literal
    ("tiny", "f32", 0, 2, 3, 1, 5, 17, False),
    ("tiny", "f32", 0, 2, 3, 2, 5, 17, True),
    ("tiny", "f32", 1, 1, 2, 1, 1, 12, False),        # P = 1: the mask of Eq. 3 as printed, p mod tau = 0
    ("mid", "bf16", 0, 2, 3, 2, 11, 40, False),
    ("mid", "bf16", 2, 2, 4, 1, 9, 30, False),
    ("tiny", "bf16", 0, 2, 3, 1, 7, 300, False),      # longer than one chunk of the workspace
]


@pytest.mark.parametrize("shape_name,dtype,L_e,L_d,tau,B,P,n,literal", MASKED_CASES)
def test_masked_parallel_forward(dmtd, shape_name, dtype, L_e, L_d, tau, B, P, n, literal):
    """Eq. 1-5 as one pass on the GPU against the oracle's, every position from P-1 on."""
    shape = SHAPES[shape_name].with_(dtype=dtype)
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    tokens = make_prompts(shape.vocab, B, n, seed=5).numpy()
    eng = dmtd.Dmtd(shape, to_cuda(w), L_d=L_d, tau=tau, max_batch=B, max_seq=n + 2, kv_dtype="f32")
    eng.set_option("encoding_layers", L_e)
    eng.set_option("literal_sum", int(literal))
    got = eng.masked_forward(torch.from_numpy(tokens).cuda(), P).double().cpu().numpy()
    for b in range(B):
        ref = oracle.masked_parallel_forward(shape, w, L_d, tau, tokens[b], P, literal_sum=literal, L_e=L_e)
        err = np.abs(got[b] - ref).max()
        assert err < 1e-3, err
    # the context is still without a sequence and can go on to an ordinary generation
    assert eng.state()["n_known"] == 0
    eng.prefill(torch.from_numpy(np.ascontiguousarray(tokens[:, :P])).cuda())


def test_masked_forward_equals_scheduled_decode_on_the_gpu(dmtd):
    """The GPU's two formulations against each other: teacher-forced scheduled decode (cache,
    cyclical refilling) and the one-pass masked forward over the same tokens."""
    shape = SHAPES["mid"]
    w = to_cuda(make_weights(shape, seed=0, norm_jitter=0.1))
    B, P, n_new, L_d, tau = 2, 10, 14, 2, 3
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, n_new, seed=2).numpy()
    eng = dmtd.Dmtd(shape, w, L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 2, kv_dtype="f32")
    sched, _ = gpu_forced(eng, prompts, forced)                      # [n_new, B, V]
    eng.reset()
    seq = np.concatenate([prompts, forced[:, :n_new - 1]], 1).astype(np.int32)
    one = eng.masked_forward(torch.from_numpy(np.ascontiguousarray(seq)).cuda(), P).double().cpu().numpy()   # [B, n_new, V]
    assert np.abs(one.transpose(1, 0, 2) - sched).max() < 1e-3
    from paper_2510_11958_b200.binding import STATUS
    eng.prefill(torch.from_numpy(prompts).cuda())
    with pytest.raises(dmtd.DmtdError) as e:
        eng.masked_forward(torch.from_numpy(np.ascontiguousarray(seq)).cuda(), P)
    assert e.value.status == STATUS["STATE"]


def _gumbel_noise(V, seed, position, sequence):
    """Noise of the sampling rule for one (position, sequence), vectorised: Philox4x32-10 with
    counter (i / 4, position, sequence, 0), word i mod 4, top 24 bits."""
    m32 = np.uint64(0xFFFFFFFF)
    c = [np.arange((V + 3) // 4, dtype=np.uint64), np.full((V + 3) // 4, position, np.uint64),
         np.full((V + 3) // 4, sequence, np.uint64), np.zeros((V + 3) // 4, np.uint64)]
    k0, k1 = np.uint64(seed & 0xFFFFFFFF), np.uint64(seed >> 32)
    for _ in range(10):
        p0, p1 = np.uint64(0xD2511F53) * c[0], np.uint64(0xCD9E8D57) * c[2]
        c = [(p1 >> np.uint64(32)) ^ c[1] ^ k0, p1 & m32, (p0 >> np.uint64(32)) ^ c[3] ^ k1, p0 & m32]
        k0, k1 = (k0 + np.uint64(0x9E3779B9)) & m32, (k1 + np.uint64(0xBB67AE85)) & m32
    words = np.stack(c, 1).reshape(-1)[:V]
    u = ((words >> np.uint64(8)).astype(np.float64) + 0.5) / 16777216.0
    return -np.log(-np.log(u))


@pytest.mark.parametrize("B,fused", [(1, 1), (1, 0), (3, 1)])
def test_sampling_matches_oracle_draws(dmtd, B, fused):
    """Tokens drawn from softmax(logits / T) inside the fused pick (pass kernel at batch 1, per-step
    kernels otherwise): teacher-forced, the model's own draw at every pass against the oracle's
    wherever the oracle's decision (logit / T + noise) has a clear margin; the noise is a function
    of (seed, position, sequence, index) alone, so both sides see the same."""
    shape = SHAPES["mid"]
    w = make_weights(shape, seed=0, norm_jitter=0.1)
    P, n_new, L_d, tau, T, seed = 12, 13, 2, 3, 0.8, 0x1234567887654321
    prompts = make_prompts(shape.vocab, B, P, seed=1).numpy()
    forced = make_prompts(shape.vocab, B, n_new, seed=2).numpy()
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 1)
    o.set_sampling(T, seed)
    tok, lg = o.prefill(prompts, forced_first=forced[:, 0])
    l, am = o.decode_forced(np.ascontiguousarray(forced[:, 1:]))
    ref_logits, ref_draw = np.concatenate([lg[None], l], 0), np.concatenate([tok[None], am], 0)
    eng = dmtd.Dmtd(shape, to_cuda(w), L_d=L_d, tau=tau, max_batch=B, max_seq=P + n_new + 1, kv_dtype="f32")
    eng.set_option("fused_pass", fused)
    eng.set_sampling(T, seed)
    got_logits, got_draw = gpu_forced(eng, prompts, forced)
    assert np.abs(got_logits - ref_logits).max() < 1e-3
    n_clear = 0
    for i in range(n_new):
        for b in range(B):
            v = ref_logits[i, b] / T + _gumbel_noise(shape.vocab, seed, P + i, b)
            assert int(np.argmax(v)) == ref_draw[i, b]           # the test's restatement agrees with the oracle
            top = np.sort(v)[-2:]
            if top[1] - top[0] > 5e-2:
                n_clear += 1
                assert got_draw[i, b] == ref_draw[i, b]
    assert n_clear >= n_new * B // 2
    greedy = ref_logits.argmax(-1)
    assert (ref_draw != greedy).any()                            # the draws are not the greedy picks
    assert eng.device_state() == o.state()


def test_sampling_free_running_is_reproducible(dmtd):
    shape = SHAPES["mid"]
    w = to_cuda(make_weights(shape, seed=0))
    prompts = torch.from_numpy(make_prompts(shape.vocab, 1, 10, seed=1).numpy()).cuda()
    runs = []
    for seed in (7, 7, 8):
        eng = dmtd.Dmtd(shape, w, L_d=2, tau=3, max_batch=1, max_seq=40, kv_dtype="f32")
        eng.set_sampling(1.0, seed)
        eng.prefill(prompts)
        toks = []
        for _ in range(5):
            rc, n, out = eng.decode_cycle(3)
            toks.append(out[:, :n].clone())
        runs.append(torch.cat(toks, 1).cpu())
    assert (runs[0] == runs[1]).all() and (runs[0] != runs[2]).any()

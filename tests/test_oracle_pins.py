"""Pins of the CPU oracle against things other than itself.

Each test names the mistake it is there to catch.  Library routines used as references:
torch's rms_norm / silu / scaled_dot_product_attention / matmul, and the `transformers`
implementation of the Qwen3 decoder (the base model named in Section 3.1 of the paper).
"""
import math
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from synthetic import SHAPES, make_weights, make_prompts

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
TINY = SHAPES["tiny"]


# ----------------------------------------------------------------------------- unit functions

def test_rmsnorm_matches_library(oracle_lib):
    g = torch.Generator().manual_seed(3)
    x = torch.randn(5, 96, generator=g, dtype=torch.float64) * 3.0
    w = torch.randn(96, generator=g, dtype=torch.float64)
    ref = F.rms_norm(x, (96,), w, eps=1e-6).numpy()
    got = oracle_lib.rmsnorm(x.numpy(), w.numpy(), 1e-6)
    np.testing.assert_allclose(got, ref, rtol=1e-13, atol=1e-13)
    # unit weights: output has RMS 1 (eps negligible)
    y = oracle_lib.rmsnorm(x.numpy(), np.ones(96), 1e-12)
    np.testing.assert_allclose(np.sqrt((y ** 2).mean(-1)), 1.0, rtol=1e-9)


def test_silu_matches_library(oracle_lib):
    for t in (-20.0, -3.0, -0.5, 0.0, 0.7, 4.0, 30.0):
        assert oracle_lib.silu(t) == pytest.approx(F.silu(torch.tensor(t, dtype=torch.float64)).item(),
                                                   rel=1e-14, abs=1e-300)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_linear_is_x_times_w_transposed(oracle_lib, dtype):
    # catches a transposed operand and a wrong bf16 widening
    g = torch.Generator().manual_seed(4)
    W = torch.randn(37, 53, generator=g).to(dtype)
    x = torch.randn(3, 53, generator=g, dtype=torch.float64)
    ref = (x @ W.double().T).numpy()
    np.testing.assert_allclose(oracle_lib.linear(W, x.numpy()), ref, rtol=1e-12, atol=1e-12)


def test_rope_closed_forms(oracle_lib):
    theta = 1.0e4
    # position 0 is the identity
    v = np.arange(1.0, 9.0)
    np.testing.assert_array_equal(oracle_lib.rope(v, 0, theta), v)
    # d = 2: one pair, frequency theta^0 = 1, so (1, 0) turns by `pos` radians
    np.testing.assert_allclose(oracle_lib.rope(np.array([1.0, 0.0]), 2, theta),
                               [math.cos(2.0), math.sin(2.0)], atol=1e-15)
    # d = 4: pairs are (0, 2) and (1, 3); pair 1 turns at theta^(-2/4) = 0.01 rad per position
    out = oracle_lib.rope(np.array([0.0, 1.0, 0.0, 0.0]), 100, theta)
    np.testing.assert_allclose(out, [0.0, math.cos(1.0), 0.0, math.sin(1.0)], atol=1e-14)
    # each pair keeps its norm
    g = np.random.default_rng(0)
    v = g.standard_normal(64)
    r = oracle_lib.rope(v, 1234, 1.0e6)
    np.testing.assert_allclose(v[:32] ** 2 + v[32:] ** 2, r[:32] ** 2 + r[32:] ** 2, rtol=1e-12)
    # the score of a rotated pair depends on the distance only
    q, k = g.standard_normal(64), g.standard_normal(64)
    a = oracle_lib.rope(q, 17, 1e6) @ oracle_lib.rope(k, 5, 1e6)
    b = oracle_lib.rope(q, 1012, 1e6) @ oracle_lib.rope(k, 1000, 1e6)
    assert a == pytest.approx(b, rel=1e-10)


def _brute_force_attention(q, k, v, pos0):
    """softmax(Q K^T / sqrt(d) + causal mask) V with dense matrices, one head at a time."""
    R, nq, d = q.shape
    nkv = k.shape[1]
    n = pos0 + R
    out = np.zeros_like(q)
    for h in range(nq):
        kh = k[:, h // (nq // nkv), :]
        vh = v[:, h // (nq // nkv), :]
        S = q[:, h, :] @ kh.T / math.sqrt(d)                      # [R, n]
        mask = np.arange(n)[None, :] > (pos0 + np.arange(R))[:, None]
        S = np.where(mask, -np.inf, S)
        Pm = np.exp(S - S.max(-1, keepdims=True))
        Pm /= Pm.sum(-1, keepdims=True)
        out[:, h, :] = Pm @ vh
    return out


@pytest.mark.parametrize("R,pos0,nq,nkv,d", [(1, 0, 4, 2, 8), (1, 9, 4, 2, 8), (3, 5, 8, 2, 16),
                                             (4, 0, 4, 4, 8), (7, 3, 6, 1, 4)])
def test_attention_brute_force_and_library(oracle_lib, R, pos0, nq, nkv, d):
    g = np.random.default_rng(R * 100 + pos0)
    n = pos0 + R
    q = g.standard_normal((R, nq, d))
    k = g.standard_normal((n, nkv, d))
    v = g.standard_normal((n, nkv, d))
    got = oracle_lib.attention(q, k, v, pos0)
    np.testing.assert_allclose(got, _brute_force_attention(q, k, v, pos0), rtol=1e-11, atol=1e-12)
    # library routine: expand KV heads, boolean causal mask offset by pos0
    tq = torch.from_numpy(q).permute(1, 0, 2)[None]                       # [1, nq, R, d]
    tk = torch.from_numpy(k).permute(1, 0, 2).repeat_interleave(nq // nkv, 0)[None]
    tv = torch.from_numpy(v).permute(1, 0, 2).repeat_interleave(nq // nkv, 0)[None]
    allowed = torch.arange(n)[None, :] <= (pos0 + torch.arange(R))[:, None]
    ref = F.scaled_dot_product_attention(tq, tk, tv, attn_mask=allowed)[0].permute(1, 0, 2)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-10, atol=1e-12)


def test_attention_uniform_when_query_is_zero(oracle_lib):
    # closed form: q = 0 gives equal weights, so the output is the running mean of V
    n, nkv, d = 6, 2, 4
    g = np.random.default_rng(1)
    v = g.standard_normal((n, nkv, d))
    k = g.standard_normal((n, nkv, d))
    out = oracle_lib.attention(np.zeros((n, 2, d)), k, v, 0)
    for r in range(n):
        np.testing.assert_allclose(out[r], v[: r + 1].mean(0), rtol=1e-12, atol=1e-14)


# ----------------------------------------------------------------------------- whole model vs a library

def _hf_model(shape, weights):
    from transformers import Qwen3Config, Qwen3ForCausalLM
    cfg = Qwen3Config(vocab_size=shape.vocab, hidden_size=shape.hidden,
                      intermediate_size=shape.intermediate, num_hidden_layers=shape.n_layers,
                      num_attention_heads=shape.n_q_heads, num_key_value_heads=shape.n_kv_heads,
                      head_dim=shape.head_dim, rope_theta=shape.rope_theta,
                      rms_norm_eps=shape.rms_eps, tie_word_embeddings=True, attention_bias=False,
                      max_position_embeddings=4096, attn_implementation="eager")
    m = Qwen3ForCausalLM(cfg).double().eval()
    sd = {"model.embed_tokens.weight": weights["embed"], "model.norm.weight": weights["final_norm"],
          "lm_head.weight": weights["embed"]}
    names = {"input_norm": "input_layernorm", "post_norm": "post_attention_layernorm",
             "q_proj": "self_attn.q_proj", "k_proj": "self_attn.k_proj", "v_proj": "self_attn.v_proj",
             "o_proj": "self_attn.o_proj", "q_norm": "self_attn.q_norm", "k_norm": "self_attn.k_norm",
             "gate_proj": "mlp.gate_proj", "up_proj": "mlp.up_proj", "down_proj": "mlp.down_proj"}
    for i, lw in enumerate(weights["layers"]):
        for k, v in lw.items():
            sd[f"model.layers.{i}.{names[k]}.weight"] = v
    missing, unexpected = m.load_state_dict({k: v.double() for k, v in sd.items()}, strict=False)
    assert not unexpected, unexpected
    assert all("rotary" in k or "inv_freq" in k for k in missing), missing
    return m


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_block_definition_matches_library_qwen3(dtype):
    """The oracle's decoder block (norms, QK-norm, RoPE pairing, GQA, SwiGLU, tied head) against
    the `transformers` Qwen3 model on the same weights: catches any wrong reading of the block."""
    shape = TINY.with_(dtype=dtype)
    w = make_weights(shape, seed=0, std=0.05, norm_jitter=0.2)
    prompt = make_prompts(shape.vocab, 1, 12, seed=1)[0].numpy()
    n_new = 5
    toks, logits, am = oracle.vanilla_generate(shape, w, prompt, n_new)
    m = _hf_model(shape, w)
    with torch.no_grad():
        ref = m(torch.from_numpy(toks[:-1].astype(np.int64))[None]).logits[0].numpy()
    # logits after position P-1+i predict token P+i
    P = prompt.size
    # the library computes its rotary cos/sin table in fp32 even for a double model, which
    # limits the agreement to ~1e-6; a wrong reading of the block shows up at 1e-2 .. 1
    np.testing.assert_allclose(logits, ref[P - 1:], rtol=0, atol=1e-5)
    assert np.abs(logits).max() > 0.5
    assert (toks[P:] == ref[P - 1:].argmax(-1)).all()


def test_identity_layers_closed_form():
    """o_proj = down_proj = 0 turns every layer into the identity, so the logits are
    rmsnorm(E[tok]) * w_f @ E^T regardless of tau and L_d."""
    shape = TINY
    w = make_weights(shape, seed=2, norm_jitter=0.1)
    for lw in w["layers"]:
        lw["o_proj"].zero_()
        lw["down_proj"].zero_()
    prompt = make_prompts(shape.vocab, 1, 7, seed=5)
    o = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=32)
    tok, logits = o.prefill(prompt.numpy())
    E = w["embed"].double().numpy()
    for step in range(6):
        last = prompt[0, -1].item() if step == 0 else prev
        x = E[last]
        a = x / math.sqrt((x ** 2).mean() + shape.rms_eps) * w["final_norm"].double().numpy()
        np.testing.assert_allclose(logits[0], a @ E.T, rtol=1e-11, atol=1e-13)
        prev = int(tok[0])
        rc, t, lg = o.decode_cycle(1)
        tok, logits = t[:, 0], lg[0]


# ----------------------------------------------------------------------------- the schedule

def _read_trace():
    rows = []
    for line in open(os.path.join(GOLDEN, "fig3_trace.txt")):
        if line.startswith("#") or not line.strip():
            continue
        idx, kind, lo, up = line.split()
        rng = lambda s: None if s == "-" else tuple(int(t) for t in s.split("-"))
        rows.append((int(idx), kind, rng(lo), rng(up)))
    return rows


def test_fig3_worked_example_trace():
    """Section 2.2's example: which positions enter the lower / upper layers in passes 1-7."""
    shape = TINY
    w = make_weights(shape, seed=0)
    o = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=32)
    o.prefill(make_prompts(shape.vocab, 1, 5, seed=1).numpy())
    for _ in range(3):
        o.decode_cycle(3, want_logits=False)
    kinds = {0: "prefill", 1: "full", 2: "upper"}
    tr = o.trace()
    golden = _read_trace()
    assert len(tr) >= len(golden)
    for (idx, kind, lo, up), rec in zip(golden, tr):
        assert kinds[rec["kind"]] == kind, idx
        got_lo = None if rec["lo_begin"] == rec["lo_end"] else (rec["lo_begin"], rec["lo_end"] - 1)
        got_up = (rec["up_begin"], rec["up_end"] - 1)
        assert got_lo == lo, (idx, got_lo, lo)
        assert got_up == up, (idx, got_up, up)


def test_mask_pattern_of_eq3(oracle_lib):
    # the paper's pattern for tau = 3 is [1,0,0,1,0,0,...] (anchor at position 0 <=> P = 1)
    assert [oracle_lib.anchor_mask(p, 1, 3) for p in range(9)] == [1, 0, 0, 1, 0, 0, 1, 0, 0]
    # anchored at the last prompt token (P = 5): prompt all ones, then positions 4, 7, 10
    assert [oracle_lib.anchor_mask(p, 5, 3) for p in range(12)] == [1] * 5 + [0, 0, 1, 0, 0, 1, 0]


def test_plt_printed_values(oracle_lib):
    for line in open(os.path.join(GOLDEN, "plt_values.txt")):
        if line.startswith("#") or not line.strip():
            continue
        L, L_d, tau, val, dec, what = line.split()
        v = oracle_lib.plt(int(L), int(L_d), int(tau))
        v = 1.0 / v if what == "inverse" else v
        assert round(v, int(dec)) == float(val)
    assert oracle_lib.plt(36, 8, 2) == pytest.approx(22 / 36)
    assert oracle_lib.plt(36, 8, 4) == pytest.approx(60 / 144)
    # second form of Eq. 7
    for L, L_d, tau in ((36, 8, 3), (28, 4, 6), (4, 2, 3)):
        assert oracle_lib.plt(L, L_d, tau) == pytest.approx(1 / tau + (tau - 1) / tau * L_d / L)


@pytest.mark.parametrize("tau,L_d", [(3, 2), (2, 1), (4, 3), (1, 2)])
def test_layer_counters_give_plt(oracle_lib, tau, L_d):
    """Per steady cycle: one pass over all L layers plus tau-1 passes over the L_d upper layers;
    over a run every token visits every layer exactly once (same total load as vanilla)."""
    shape = TINY
    L = shape.n_layers
    w = make_weights(shape, seed=0)
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_seq=64)
    P = 6
    o.prefill(make_prompts(shape.vocab, 1, P, seed=1).numpy(), want_logits=False)
    if tau > 1:
        o.decode_cycle(tau, want_logits=False)       # finish cycle 1 (tau-1 upper-only passes)
    c0, r0 = o.layer_counters()
    n_cycles = 4
    for _ in range(n_cycles):
        rc, toks, _ = o.decode_cycle(tau, want_logits=False)
        assert rc == 0 and toks.shape[1] == tau
    c1, r1 = o.layer_counters()
    calls = (c1 - c0).sum()
    assert calls == n_cycles * (L + (tau - 1) * L_d)
    assert calls / (n_cycles * tau * L) == pytest.approx(oracle_lib.plt(L, L_d, tau))
    lower, upper = slice(0, L - L_d), slice(L - L_d, L)
    assert ((c1 - c0)[lower] == n_cycles).all() and ((r1 - r0)[lower] == n_cycles * tau).all()
    assert ((c1 - c0)[upper] == n_cycles * tau).all() and ((r1 - r0)[upper] == n_cycles * tau).all()
    st = o.state()
    assert st["n_known"] == P + 1 + (tau - 1) + n_cycles * tau
    assert st["n_emitted"] == st["n_known"] - P
    assert st["slot"] == 0 and st["cycle"] == 1 + n_cycles
    assert st["up_len"] == st["n_known"] - 1 and st["lo_len"] == st["n_known"] - tau


def test_state_after_each_pass():
    shape = TINY
    w = make_weights(shape, seed=0)
    tau, P = 3, 5
    o = oracle.Oracle(shape, w, L_d=2, tau=tau, max_seq=64)
    o.prefill(make_prompts(shape.vocab, 1, P, seed=1).numpy(), want_logits=False)
    assert o.state() == dict(n_known=6, lo_len=5, up_len=5, cycle=1, slot=1, n_emitted=1, tau=3, L_d=2)
    o.decode_cycle(1, want_logits=False)
    assert o.state() == dict(n_known=7, lo_len=5, up_len=6, cycle=1, slot=2, n_emitted=2, tau=3, L_d=2)
    o.decode_cycle(5, want_logits=False)              # stops at the cycle boundary
    assert o.state() == dict(n_known=8, lo_len=5, up_len=7, cycle=1, slot=0, n_emitted=3, tau=3, L_d=2)
    o.decode_cycle(1, want_logits=False)              # full pass, truncated by max_new
    assert o.state() == dict(n_known=9, lo_len=8, up_len=8, cycle=2, slot=1, n_emitted=4, tau=3, L_d=2)


def test_capacity_and_order_errors():
    shape = TINY
    w = make_weights(shape, seed=0)
    o = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=8)
    rc, _, _ = o.decode_cycle(3, want_logits=False)
    assert rc == -3                                  # decode before prefill
    o.prefill(make_prompts(shape.vocab, 1, 5, seed=1).numpy(), want_logits=False)
    rc, toks, _ = o.decode_cycle(3, want_logits=False)
    assert rc == 0 and toks.shape[1] == 2
    rc, toks, _ = o.decode_cycle(3, want_logits=False)   # positions 8.. do not fit
    assert rc == -4 and toks.shape[1] == 0
    with pytest.raises(ValueError):
        oracle.Oracle(shape, w, L_d=5, tau=3)
    with pytest.raises(ValueError):
        oracle.Oracle(shape, w, L_d=2, tau=0)


# ----------------------------------------------------------------------------- special cases of the whole

def _run_dmtd(shape, w, L_d, tau, prompt, n_new, forced=None, max_batch=1, literal_sum=False):
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_batch=max_batch, max_seq=prompt.shape[1] + n_new + 1,
                      literal_sum=literal_sum)
    tok, lg = o.prefill(prompt, forced_first=None if forced is None else forced[:, 0])
    toks, logits = [tok], [lg]
    if forced is None:
        while len(toks) < n_new:
            rc, t, l = o.decode_cycle(n_new - len(toks))
            assert rc == 0
            toks += [t[:, i] for i in range(t.shape[1])]
            logits += [l[i] for i in range(l.shape[0])]
    else:
        l, am = o.decode_forced(forced[:, 1:n_new])
        toks += [am[i] for i in range(am.shape[0])]
        logits += [l[i] for i in range(l.shape[0])]
    return np.stack(toks, 1), np.stack(logits, 0), o           # [B, n], [n, B, V]


def test_tau1_is_vanilla_decoding():
    """tau = 1 must reproduce plain full-depth autoregressive decoding token for token."""
    shape = TINY
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 1, 32, seed=1).numpy()
    n_new = 24
    toks, logits, _ = _run_dmtd(shape, w, 2, 1, prompt, n_new)
    vt, vl, _ = oracle.vanilla_generate(shape, w, prompt[0], n_new)
    assert (toks[0] == vt[32:]).all()
    np.testing.assert_allclose(logits[:, 0], vl, rtol=0, atol=1e-12)


@pytest.mark.parametrize("tau", [2, 3, 4])
def test_all_layers_decoding_is_vanilla(tau):
    """L_d = L: the lower range is empty, every pass is full depth, for any tau."""
    shape = TINY
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 1, 9, seed=1).numpy()
    n_new = 10
    toks, logits, _ = _run_dmtd(shape, w, shape.n_layers, tau, prompt, n_new)
    vt, vl, _ = oracle.vanilla_generate(shape, w, prompt[0], n_new)
    assert (toks[0] == vt[9:]).all()
    np.testing.assert_allclose(logits[:, 0], vl, rtol=0, atol=1e-12)


def test_dmtd_differs_from_vanilla_when_tau_gt_1():
    # sanity of the two tests above: the schedule is not a no-op
    shape = TINY
    w = make_weights(shape, seed=0, std=0.05)
    prompt = make_prompts(shape.vocab, 1, 9, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, 8, seed=7).numpy()
    _, lg, _ = _run_dmtd(shape, w, 2, 3, prompt, 8, forced=forced)
    _, vl, _ = oracle.vanilla_generate(shape, w, prompt[0], 8, forced=forced[0])
    d = np.abs(lg[:, 0] - vl).max(-1)
    assert d[0] < 1e-12                      # prefill row is full depth
    assert d[1] > 1e-3 and d[2] > 1e-3       # upper-only passes see an embedding, not h_think
    assert d[3] > 1e-6                       # full pass, but the upper KV of 2 positions differs


@pytest.mark.parametrize("tau,L_d,P", [(3, 2, 5), (2, 1, 4), (4, 3, 7), (3, 4, 6)])
@pytest.mark.parametrize("literal", [False, True])
def test_scheduled_equals_masked_parallel_forward(tau, L_d, P, literal):
    """Section 2.2's cached, pass-by-pass schedule computes the same function as one masked
    parallel forward (Eq. 1-5) over the final sequence."""
    shape = TINY
    w = make_weights(shape, seed=3, std=0.05, norm_jitter=0.1)
    prompt = make_prompts(shape.vocab, 1, P, seed=2).numpy()
    n_new = 11
    forced = make_prompts(shape.vocab, 1, n_new, seed=9).numpy()
    _, logits, _ = _run_dmtd(shape, w, L_d, tau, prompt, n_new, forced=forced, literal_sum=literal)
    seq = np.concatenate([prompt[0], forced[0, : n_new - 1]])
    ref = oracle.masked_parallel_forward(shape, w, L_d, tau, seq, P, literal_sum=literal)
    np.testing.assert_allclose(logits[:, 0], ref, rtol=0, atol=1e-11)


def test_batch_independence():
    shape = TINY
    w = make_weights(shape, seed=0)
    prompts = make_prompts(shape.vocab, 3, 6, seed=4).numpy()
    toks, logits, _ = _run_dmtd(shape, w, 2, 3, prompts, 7, max_batch=3)
    for b in range(3):
        tb, lb, _ = _run_dmtd(shape, w, 2, 3, prompts[b:b + 1], 7)
        assert (tb[0] == toks[b]).all()
        np.testing.assert_array_equal(lb[:, 0], logits[:, b])


def test_step_layers_matches_pass():
    """step_layers over all layers on the embeddings of a prompt = what prefill caches."""
    shape = TINY
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 1, 6, seed=1).numpy()
    a = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=16)
    a.prefill(prompt, want_logits=False)
    b = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=16)
    x = w["embed"].double().numpy()[prompt[0]][None]
    b.step_layers(0, shape.n_layers, x, 0)
    for l in range(shape.n_layers):
        ka, va = a.kv_cache(l, 0, 6)
        kb, vb = b.kv_cache(l, 0, 6)
        np.testing.assert_array_equal(ka, kb)
        np.testing.assert_array_equal(va, vb)


# ----------------------------------------------------------------------------- corners named by review

def test_chunked_prefill_equals_unchunked_forward():
    """The prefill feeds prompts longer than 256 rows in causal chunks; a wrong chunk origin (rows
    of the second chunk rotated or cached at the first chunk's positions) would pass every pin
    with a short prompt.  The no-cache, no-chunk forward over the same 300 tokens must give the
    same logits for the first generated token."""
    shape = TINY
    w = make_weights(shape, seed=4, norm_jitter=0.1)
    P = 300
    prompt = make_prompts(shape.vocab, 1, P, seed=9).numpy()
    o = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=P + 4)
    tok, logits = o.prefill(prompt)
    vt, vl, vam = oracle.vanilla_generate(shape, w, prompt[0], 1)
    np.testing.assert_allclose(logits[0], vl[0], rtol=0, atol=1e-11)
    assert int(tok[0]) == int(vam[0])
    # and the cache rows of the second chunk sit at their own positions: one more (short) pass
    # through the decoding layers reads them
    rc, t, lg = o.decode_cycle(1)
    seq = np.concatenate([prompt[0], tok]).astype(np.int32)
    ref = oracle.masked_parallel_forward(shape, w, 2, 3, seq, P)
    np.testing.assert_allclose(lg[0, 0], ref[1], rtol=0, atol=1e-11)


def test_argmax_picks_lowest_index_on_exact_tie():
    """Two identical embedding rows give bit-identical logits at their two vocabulary entries
    (identity layers: o_proj = down_proj = 0).  Make that pair the maximum: the lower index
    must be emitted.  `>=` in place of `>` in the pick would emit the higher one."""
    shape = TINY
    w = make_weights(shape, seed=2)
    for lw in w["layers"]:
        lw["o_proj"].zero_()
        lw["down_proj"].zero_()
    lo, hi, last = 17, 801, 5
    # logits = rmsnorm(E[last]) . E[v]: the row parallel to E[last] with a large norm wins
    w["embed"][lo] = 3.0 * w["embed"][last]
    w["embed"][hi] = w["embed"][lo]
    prompt = np.array([[9, 3, last]], np.int32)
    o = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=16)
    tok, logits = o.prefill(prompt)
    assert logits[0, lo] == logits[0, hi] == logits[0].max()
    assert int(tok[0]) == lo
    # the same through a decode pass
    w2 = {"embed": w["embed"].clone(), "final_norm": w["final_norm"], "layers": w["layers"]}
    o2 = oracle.Oracle(shape, w2, L_d=2, tau=3, max_seq=16)
    o2.prefill(prompt, forced_first=np.array([last], np.int32))
    rc, t, lg = o2.decode_cycle(1)
    assert lg[0, 0, lo] == lg[0, 0, hi] == lg[0, 0].max()
    assert int(t[0, 0]) == lo


def test_set_tau_after_prefill_at_cycle_boundary():
    """The cycle length may change between cycles (Section 3.7 evaluates inference cycle lengths
    other than the training one).  A change in mid-cycle is refused; after a change at a boundary
    the next full pass still refills every pending position of the old cycle, and the cycles that
    follow have the new length: the pass trace says which positions enter which layers."""
    shape = TINY
    w = make_weights(shape, seed=0)
    P = 6
    prompt = make_prompts(shape.vocab, 1, P, seed=1).numpy()
    o = oracle.Oracle(shape, w, L_d=2, tau=3, max_seq=40)
    o.prefill(prompt)
    assert o.set_tau(2) == -3                   # mid-cycle: refused
    o.decode_cycle(3)                           # finishes cycle 1 (2 short passes)
    assert o.state()["slot"] == 0
    assert o.set_tau(2) == 0
    st = o.state()
    assert st["tau"] == 2 and st["n_known"] == P + 3
    rc, t, lg = o.decode_cycle(2)
    assert rc == 0 and t.shape[1] == 2
    tr = o.trace()
    # pass 3: full pass refills the two pending positions and the newest, then one short pass
    assert (tr[3]["kind"], tr[3]["lo_begin"], tr[3]["lo_end"], tr[3]["up_begin"]) == (1, P, P + 3, P + 2)
    assert (tr[4]["kind"], tr[4]["up_begin"]) == (2, P + 3)
    rc, t2, lg2 = o.decode_cycle(2)
    tr = o.trace()
    assert (tr[5]["kind"], tr[5]["lo_begin"], tr[5]["lo_end"]) == (1, P + 3, P + 5)
    st = o.state()
    assert st["cycle"] == 3 and st["lo_len"] == P + 5 and st["slot"] == 0


# ----------------------------------------------------------------------------- ExDy (encoding layers reused too)

def _run_exdy(shape, w, L_e, L_d, tau, prompt, forced, literal=False):
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_seq=prompt.shape[1] + forced.shape[1] + 1,
                      literal_sum=literal, L_e=L_e)
    tok, lg = o.prefill(prompt, forced_first=forced[:, 0])
    l, am = o.decode_forced(forced[:, 1:])
    return np.concatenate([lg[None], l], 0), o


@pytest.mark.parametrize("L_e,L_d,tau,P", [(1, 1, 3, 5), (1, 2, 2, 4), (2, 1, 4, 7), (1, 1, 1, 3)])
@pytest.mark.parametrize("literal", [False, True])
def test_exdy_scheduled_equals_masked_parallel_forward(L_e, L_d, tau, P, literal):
    """Section 2.1 (after Eq. 4): with the encoding layers reused, h_enc takes h_emb's place in
    Eq. 4.  The cached, scheduled decode (encoding + decoding layers on every short pass, the
    thinking layers refilled from the saved h_enc rows) must equal the one-shot masked forward
    written from Eq. 1-5.  A refill fed with embeddings instead of h_enc, a short pass that skips
    the encoding layers, or encoding-layer KV missing at some position each break the equality."""
    shape = TINY
    w = make_weights(shape, seed=6, norm_jitter=0.1)
    n_new = 3 * tau + 2
    prompt = make_prompts(shape.vocab, 1, P, seed=3).numpy()
    forced = make_prompts(shape.vocab, 1, n_new, seed=4).numpy()
    logits, o = _run_exdy(shape, w, L_e, L_d, tau, prompt, forced, literal)
    seq = np.concatenate([prompt[0], forced[0]]).astype(np.int32)
    ref = oracle.masked_parallel_forward(shape, w, L_d, tau, seq[:P + n_new - 1], P, literal_sum=literal, L_e=L_e)
    np.testing.assert_allclose(logits[:, 0], ref, rtol=0, atol=1e-11)


def test_exdy_with_no_thinking_layers_is_vanilla_decoding():
    """L_e + L_d = L: nothing is left to skip, every pass runs every layer on one row."""
    shape = TINY
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 1, 9, seed=1).numpy()
    n_new = 10
    o = oracle.Oracle(shape, w, L_d=3, tau=3, max_seq=32, L_e=1)
    tok, lg = o.prefill(prompt)
    toks, logits = [tok], [lg]
    while len(toks) < n_new:
        rc, t, l = o.decode_cycle(n_new - len(toks))
        toks += [t[:, i] for i in range(t.shape[1])]
        logits += [l[i] for i in range(l.shape[0])]
    vt, vl, _ = oracle.vanilla_generate(shape, w, prompt[0], n_new)
    assert (np.stack(toks, 1)[0] == vt[9:]).all()
    np.testing.assert_allclose(np.stack(logits, 0)[:, 0], vl, rtol=0, atol=1e-12)


@pytest.mark.parametrize("L_e,L_d,tau", [(1, 1, 3), (1, 2, 2), (2, 1, 4)])
def test_exdy_layer_counters(oracle_lib, L_e, L_d, tau):
    """Layers traversed per cycle: the encoding and decoding layers on every pass, the thinking
    layers once: L + (tau - 1)(L_e + L_d), i.e. Eq. 7 with L_e + L_d reused layers."""
    shape = TINY
    L = shape.n_layers
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 1, 4, seed=1).numpy()
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_seq=64, L_e=L_e)
    o.prefill(prompt, want_logits=False)
    if tau > 1:
        o.decode_cycle(tau, want_logits=False)
    c0, r0 = o.layer_counters()
    n_cycles = 3
    for _ in range(n_cycles):
        o.decode_cycle(tau, want_logits=False)
    c1, r1 = o.layer_counters()
    calls, rows = c1 - c0, r1 - r0
    for l in range(L):
        reused = l < L_e or l >= L - L_d
        assert calls[l] == n_cycles * (tau if reused else 1)
        assert rows[l] == n_cycles * tau                      # every token visits every layer once
    plt = calls.sum() / (n_cycles * tau * L)
    assert abs(plt - oracle_lib.plt(L, L_e + L_d, tau)) < 1e-15


def test_exdy_differs_from_decoding_layers_only():
    """Reusing an encoding layer changes the function (it is not a re-labelling of E0Dy)."""
    shape = TINY
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 1, 5, seed=1).numpy()
    forced = make_prompts(shape.vocab, 1, 7, seed=2).numpy()
    a, _ = _run_exdy(shape, w, 1, 1, 3, prompt, forced)
    b, _ = _run_exdy(shape, w, 0, 1, 3, prompt, forced)
    assert np.abs(a[0] - b[0]).max() == 0.0                   # the prefill is the same full-depth pass
    assert np.abs(a[1:3] - b[1:3]).max() > 1e-3               # the short passes are not


def test_exdy_rejects_bad_split():
    shape = TINY
    w = make_weights(shape, seed=0)
    with pytest.raises(ValueError):
        oracle.Oracle(shape, w, L_d=3, tau=3, L_e=2)           # 2 + 3 > 4 layers


# ----------------------------------------------------------------------------- sampling (extension beside the greedy rule)

def test_philox_known_answers(oracle_lib):
    """The counter-based generator against its published known-answer vectors: a wrong round
    constant, a swapped word or nine rounds instead of ten changes every output word."""
    n = 0
    for line in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt")):
        if line.startswith("#") or not line.strip():
            continue
        w = [int(x, 16) for x in line.split()]
        assert oracle_lib.philox(w[0:4], w[4:6]) == w[6:10]
        n += 1
    assert n == 3


def test_gumbel_max_sampling_follows_softmax(oracle_lib):
    """argmax(z / T + Gumbel noise) is a draw from softmax(z / T): over many positions the
    frequencies must match the probabilities (a missing temperature, -log(u) in place of
    -log(-log(u)), or noise shared between indices each fail by many standard deviations)."""
    z = np.array([1.0, 0.2, -0.5, 2.0, 0.0, 1.5, -1.0, 0.7])
    T, n = 0.7, 40000
    p = np.exp(z / T - (z / T).max())
    p /= p.sum()
    counts = np.zeros(z.size)
    for pos in range(n):
        counts[oracle_lib.sample_token(z, T, 1234, pos, 0)] += 1
    sigma = np.sqrt(n * p * (1 - p))
    assert (np.abs(counts - n * p) < 4.5 * sigma).all(), (counts, n * p)
    # the draw is a function of (seed, position, sequence) only
    assert oracle_lib.sample_token(z, T, 1234, 17, 0) == oracle_lib.sample_token(z, T, 1234, 17, 0)
    draws = lambda **kw: [oracle_lib.sample_token(z, T, kw.get("seed", 1), pos, kw.get("seq", 0)) for pos in range(64)]
    assert draws() != draws(seed=2) and draws() != draws(seq=1)
    # temperature 0 is the greedy rule
    assert oracle_lib.sample_token(z, 0.0, 1234, 5, 0) == 3


def test_sampled_generation_differs_from_greedy_and_keeps_the_schedule():
    shape = TINY
    w = make_weights(shape, seed=0)
    prompt = make_prompts(shape.vocab, 2, 6, seed=1).numpy()
    runs = []
    for temp in (0.0, 1.0):
        o = oracle.Oracle(shape, w, L_d=2, tau=3, max_batch=2, max_seq=32)
        o.set_sampling(temp, 99)
        tok, _ = o.prefill(prompt)
        toks = [tok]
        for _ in range(3):
            rc, t, _ = o.decode_cycle(3)
            toks += [t[:, i] for i in range(t.shape[1])]
        runs.append((np.stack(toks, 1), o.state()))
    assert runs[0][1] == runs[1][1]                       # counters do not depend on how tokens are picked
    assert (runs[0][0] != runs[1][0]).any()

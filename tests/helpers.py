"""Shared helpers of the GPU parity tests: run the oracle and the CUDA library on the same
seeded inputs.  The tolerances are the ones the build's target states: per-step logits within
2e-2 absolute, argmax equal wherever the oracle's top-2 margin exceeds 5e-2, integer
bookkeeping bit-exact."""
import numpy as np
import torch

import oracle
from synthetic import make_prompts, make_weights

LOGIT_ATOL = 2e-2
MARGIN = 5e-2


def to_cuda(weights):
    return {"embed": weights["embed"].cuda(), "final_norm": weights["final_norm"].cuda(),
            "layers": [{k: v.cuda() for k, v in lw.items()} for lw in weights["layers"]]}


def oracle_greedy(shape, w, L_d, tau, prompts, n_new, max_batch=None, literal_sum=False):
    """Free-running oracle.  Returns tokens [B, n_new], logits [n_new, B, V], states after each call."""
    B, P = prompts.shape
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_batch=max_batch or B, max_seq=P + n_new + 1,
                      literal_sum=literal_sum)
    tok, lg = o.prefill(prompts)
    toks, logits, states = [tok], [lg], [o.state()]
    while len(toks) < n_new:
        rc, t, l = o.decode_cycle(n_new - len(toks))
        assert rc == 0
        toks += [t[:, i] for i in range(t.shape[1])]
        logits += [l[i] for i in range(l.shape[0])]
        states.append(o.state())
    return np.stack(toks, 1), np.stack(logits, 0), states, o


def oracle_forced(shape, w, L_d, tau, prompts, forced, literal_sum=False):
    """Teacher-forced oracle.  forced [B, n].  Returns logits [n, B, V], argmax [n, B], oracle."""
    B, P = prompts.shape
    n = forced.shape[1]
    o = oracle.Oracle(shape, w, L_d=L_d, tau=tau, max_batch=B, max_seq=P + n + 1, literal_sum=literal_sum)
    tok, lg = o.prefill(prompts, forced_first=forced[:, 0])
    l, am = o.decode_forced(np.ascontiguousarray(forced[:, 1:]))
    return np.concatenate([lg[None], l], 0), np.concatenate([tok[None], am], 0), o


def gpu_forced(eng, prompts, forced):
    """Same through the CUDA library.  Returns logits [n, B, V] (float64 numpy), argmax [n, B]."""
    p = torch.from_numpy(np.ascontiguousarray(prompts)).cuda()
    f = torch.from_numpy(np.ascontiguousarray(forced)).cuda()
    tok, lg = eng.prefill(p, forced_first=f[:, 0].contiguous(), want_logits=True)
    logits, am = eng.decode_forced(f[:, 1:].contiguous())
    torch.cuda.synchronize()
    L = torch.cat([lg[None], logits], 0).double().cpu().numpy()
    A = torch.cat([tok[None], am], 0).cpu().numpy()
    return L, A


def check_logits(got, ref, got_argmax=None, ref_argmax=None, atol=LOGIT_ATOL):
    """got/ref [n, B, V]."""
    err = np.abs(got - ref).max()
    assert err <= atol, f"max |logit diff| {err:.3e} > {atol}"
    srt = np.sort(ref, axis=-1)
    margin = srt[..., -1] - srt[..., -2]
    clear = margin > MARGIN
    ga = got.argmax(-1) if got_argmax is None else got_argmax
    ra = ref.argmax(-1) if ref_argmax is None else ref_argmax
    assert (ga[clear] == ra[clear]).all(), "argmax differs where the oracle's margin is clear"
    return err, clear.mean()

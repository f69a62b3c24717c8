"""Seeded random weights and prompts.

Weights are N(0, std) with std = 0.02 (the 0.02 is a standard deviation), drawn in fp32 and,
for bf16 shapes, rounded to nearest-even.  Norm weights are 1 unless `norm_jitter` is given,
in which case they are 1 + norm_jitter * N(0, 1) so that a kernel that forgets a norm weight
is caught.  Every tensor gets its own generator seeded from (seed, tensor index), so the
values do not depend on the order in which tensors are requested.
"""
import torch

from .shapes import ModelShape

_LAYER_MATS = ("q_proj", "k_proj", "v_proj", "o_proj", "gate_proj", "up_proj", "down_proj")
_LAYER_NORMS = ("input_norm", "q_norm", "k_norm", "post_norm")


def _torch_dtype(shape: ModelShape):
    return {"f32": torch.float32, "bf16": torch.bfloat16}[shape.dtype]


def _mat_shape(shape: ModelShape, name: str):
    h, i = shape.hidden, shape.intermediate
    return {
        "q_proj": (shape.q_dim, h), "k_proj": (shape.kv_dim, h), "v_proj": (shape.kv_dim, h),
        "o_proj": (h, shape.q_dim), "gate_proj": (i, h), "up_proj": (i, h), "down_proj": (h, i),
    }[name]


def _norm_len(shape: ModelShape, name: str):
    return shape.head_dim if name in ("q_norm", "k_norm") else shape.hidden


def _randn(size, seed, index, device, std):
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + index) & 0x7FFFFFFFFFFFFFFF)
    return torch.randn(size, generator=g, device=device, dtype=torch.float32) * std


def make_weights(shape: ModelShape, seed: int = 0, device="cpu", std: float = 0.02,
                 norm_jitter: float = 0.0, n_layers=None):
    """Return {"embed", "final_norm", "layers": [ {name: tensor} ]} on `device`.

    Matrices are [out_features, in_features], row-major.  The LM head is tied to "embed".
    Values drawn on different devices differ (torch's generators are per device); a test
    draws once and hands the same values to both sides.
    """
    dt = _torch_dtype(shape)
    n_layers = shape.n_layers if n_layers is None else n_layers
    idx = 0

    def mat(size):
        nonlocal idx
        idx += 1
        return _randn(size, seed, idx, device, std).to(dt)

    def norm(n):
        nonlocal idx
        idx += 1
        if norm_jitter == 0.0:
            return torch.ones(n, device=device, dtype=dt)
        return (1.0 + _randn((n,), seed, idx, device, norm_jitter)).to(dt)

    out = {"embed": mat((shape.vocab, shape.hidden)), "final_norm": norm(shape.hidden),
           "layers": []}
    for _ in range(n_layers):
        lw = {}
        for name in _LAYER_MATS:
            lw[name] = mat(_mat_shape(shape, name))
        for name in _LAYER_NORMS:
            lw[name] = norm(_norm_len(shape, name))
        out["layers"].append(lw)
    return out


def make_prompts(vocab: int, batch: int, prompt_len: int, seed: int = 1):
    """Uniform random token ids, int32 [batch, prompt_len]; sequence b uses seed + b."""
    rows = []
    for b in range(batch):
        g = torch.Generator()
        g.manual_seed(seed + b)
        rows.append(torch.randint(0, vocab, (prompt_len,), generator=g, dtype=torch.int32))
    return torch.stack(rows, 0)


def weight_bytes(shape: ModelShape):
    """(bytes of one layer, bytes of the tied head) in the shape's storage type."""
    eb = 2 if shape.dtype == "bf16" else 4
    return shape.params_per_layer * eb, shape.vocab * shape.hidden * eb

"""The allocation-free attention call (dmtd_attention_decode_static) against the ordinary one.

Some users of the library cannot allocate device memory when they call it: a serving process
whose own pool already owns the GPU's free memory, or a decode loop that cannot afford the
device-wide stall of cudaMalloc / cudaFree.  For them the library keeps the attention's partial
results in a fixed built-in array.  This file checks, through the C ABI, that the variant gives
the ordinary call's result on two calls in a row (the array keeps the first call's contents
when the second one starts), and that a problem too large for the array is refused.

The file is named so that pytest collects it last: a run that stops at the first failure has
then already run every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def _case(seed, B, R, nq, nkv, D, pos0, max_seq, dtype=torch.bfloat16):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(B, R, nq, D, generator=g).cuda()
    k = torch.randn(B, nkv, max_seq, D, generator=g).to(dtype).cuda()
    v = torch.randn(B, nkv, max_seq, D, generator=g).to(dtype).cuda()
    return q, k, v, pos0


def _reference(oracle_lib, q, k, v, pos0):
    """The CPU reference attention on the same (rounded) values, sequence by sequence."""
    B, R = q.shape[0], q.shape[1]
    n = pos0 + R
    out = []
    for b in range(B):
        out.append(oracle_lib.attention(q[b].double().cpu().numpy(),
                                        k[b, :, :n].double().permute(1, 0, 2).cpu().numpy(),
                                        v[b, :, :n].double().permute(1, 0, 2).cpu().numpy(), pos0))
    return np.stack(out, 0)


def test_static_scratch_attention_matches_ordinary_call_twice(oracle_lib):
    import paper_2510_11958_b200 as pkg
    pkg.load_library()
    # the larger problem first, so that the calls after it find the array full of stale partials;
    # then row counts above one row block (more than 16 query rows per KV head: the last key slice
    # of the earlier row blocks is empty and must be skipped by the merge, not read), once with an
    # fp32 cache and once with head_dim 64 (the two other attention kernels)
    cases = [_case(21, 2, 3, 32, 8, 128, 900, 1024),
             _case(22, 1, 1, 8, 2, 128, 130, 256),
             _case(24, 2, 7, 8, 2, 128, 200, 256, torch.float32),
             _case(25, 2, 6, 8, 2, 64, 150, 192),
             _case(26, 1, 8, 8, 2, 128, 90, 128)]
    for q, k, v, pos0 in cases:
        want = pkg.attention_decode(q, k, v, pos0)
        out = torch.full_like(q, float("nan"))          # caller-owned output, allocated up front
        pkg.attention_decode_static(q, k, v, pos0, out)
        torch.cuda.synchronize()
        assert torch.isfinite(out).all()
        err = (out - want).abs().max().item()
        assert err <= 2e-5 * max(1.0, want.abs().max().item()), err
        # and directly against the CPU reference, so that this file stands on its own
        ref = _reference(oracle_lib, q, k, v, pos0)
        tol = 5e-3 if (k.dtype == torch.bfloat16 and q.shape[-1] == 128) else 2e-5
        assert np.abs(out.double().cpu().numpy() - ref).max() <= tol * max(1.0, np.abs(ref).max())


def test_static_scratch_attention_rejects_oversized_problem():
    import paper_2510_11958_b200 as pkg
    from paper_2510_11958_b200.binding import ATTENTION_STATIC_SCRATCH_BYTES, STATUS
    dll = pkg.load_library()
    B, R, nq, nkv, D, pos0, max_seq = 4, 4, 32, 8, 128, 4000, 4096
    assert dll.dmtd_attention_scratch_bytes(B, R, nq, D, pos0 + R) > ATTENTION_STATIC_SCRATCH_BYTES
    q, k, v, _ = _case(23, B, R, nq, nkv, D, pos0, max_seq)
    out = torch.zeros_like(q)
    with pytest.raises(pkg.DmtdError) as e:
        pkg.attention_decode_static(q, k, v, pos0, out)
    assert e.value.status == STATUS["CAPACITY"]
    assert (out == 0).all()                                # nothing ran

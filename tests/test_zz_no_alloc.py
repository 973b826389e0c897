"""GPU test of subgen_exact_attention_noalloc, the entry point for callers that cannot allocate.

Some users of this library run where cudaMalloc is off limits: inside a serving process whose allocator
took the device memory at start-up, or on a request path that cannot afford an allocation's device-wide
synchronisation. For them the library offers one exact-attention call whose scratch is a fixed array in
the library image. This test calls it through the C ABI twice in a row, with different shapes so that the
second call finds the first call's leftovers in the shared array, and checks both results against the
handle-based exact path (subgen_exact_append + subgen_exact_step), within the tolerances of the other
GPU tests, and on a few (sequence, head) pairs also against the CPU oracle's statement of Eq. 1. The cases
cover every branch of the kernel: several blocks per unit with the arrival counter, a single block per unit
(fewer than 64 tokens), group sizes 1, 4 and 8, both element types and both head dimensions. It is collected
last on purpose.
"""
import ctypes
import os
import sys

import pytest
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-4, torch.bfloat16: 2e-2}


def _reference(B, H, Hkv, d, n, dtype, q, K, V):
    """The existing entry points: cache the first n-1 tokens, then one exact step with the last one."""
    from paper_2402_06082_b200.binding import ExactAttention
    ex = ExactAttention(B, H, d, n, Hkv=Hkv, dtype=dtype)
    if n > 1:
        ex.append(K[:, :, : n - 1].contiguous(), V[:, :, : n - 1].contiguous())
    out = ex.step(q, K[:, :, n - 1].contiguous(), V[:, :, n - 1].contiguous())
    torch.cuda.synchronize()
    ex.close()
    return out


def _case(B, H, Hkv, d, n, dtype, seed):
    g = torch.Generator(device="cuda").manual_seed(seed)
    q = torch.randn(B, H, d, generator=g, device="cuda").to(dtype)
    K = (0.5 * torch.randn(B, Hkv, n, d, generator=g, device="cuda")).to(dtype)
    V = torch.randn(B, Hkv, n, d, generator=g, device="cuda").to(dtype)
    return q, K, V


def _rel(a, b):
    a = a.double(); b = b.double()
    return float(((a - b).norm(dim=-1) / b.norm(dim=-1).clamp_min(1e-30)).max())


def _check_against_oracle(B, H, Hkv, d, n, dtype, q, K, V, out):
    """Eq. 1 from the CPU oracle for the first and the last head of the first and the last sequence."""
    import helpers as hp
    from oracle import subgen_oracle as orc
    G = H // Hkv
    for b in sorted({0, B - 1}):
        for hq in sorted({0, H - 1}):
            want = orc.exact_attention(hp.f32(K[b, hq // G]), hp.f32(V[b, hq // G]), hp.f32(q[b, hq]))
            hp.assert_output(hp.f32(out[b, hq]), want, dtype, "no-alloc entry point vs oracle, seq %d head %d" % (b, hq))


def test_two_calls_in_a_row_match_the_handle_based_path():
    from paper_2402_06082_b200 import binding
    L = binding.load()
    cases = [(2, 8, 2, 128, 3001, torch.bfloat16, 1), (3, 4, 4, 64, 517, torch.float32, 2),
             (2, 2, 2, 128, 40, torch.bfloat16, 3),       # fewer than 64 tokens: one block per unit, no arrival counter
             (1, 16, 2, 64, 700, torch.bfloat16, 4)]      # eight query heads per KV head
    for (B, H, Hkv, d, n, dtype, seed) in cases:
        q, K, V = _case(B, H, Hkv, d, n, dtype, seed)
        out = torch.full((B, H, d), float("nan"), dtype=dtype, device="cuda")
        rc = L.subgen_exact_attention_noalloc(q.data_ptr(), K.data_ptr(), V.data_ptr(), out.data_ptr(), B, H, Hkv, d, n,
                                              binding._dtype_code(dtype), torch.cuda.current_stream().cuda_stream)
        assert rc == 0, L.subgen_last_error()
        torch.cuda.synchronize()
        want = _reference(B, H, Hkv, d, n, dtype, q, K, V)
        assert torch.isfinite(out).all()
        assert _rel(out, want) <= TOL[dtype]
        _check_against_oracle(B, H, Hkv, d, n, dtype, q, K, V, out)
    # same call again on the first shape: the array now holds the second call's leftovers
    B, H, Hkv, d, n, dtype, seed = cases[0]
    q, K, V = _case(B, H, Hkv, d, n, dtype, seed)
    out = torch.empty((B, H, d), dtype=dtype, device="cuda")
    binding.exact_attention_noalloc(q, K, V, out)
    torch.cuda.synchronize()
    assert _rel(out, _reference(B, H, Hkv, d, n, dtype, q, K, V)) <= TOL[dtype]


def test_shapes_beyond_the_fixed_scratch_are_rejected():
    from paper_2402_06082_b200 import binding
    L = binding.load()
    B, H, Hkv, d = 40, 512, 64, 128                  # 2560 units x 8 heads x 130 floats > 4 MiB
    x = torch.zeros(16, device="cuda")
    rc = L.subgen_exact_attention_noalloc(x.data_ptr(), x.data_ptr(), x.data_ptr(), x.data_ptr(), B, H, Hkv, d, 4,
                                          binding.DTYPE_BF16, None)
    assert rc == -1 and b"scratch" in L.subgen_last_error()
    rc = L.subgen_exact_attention_noalloc(None, None, None, None, 1, 1, 1, 64, 4, binding.DTYPE_BF16, None)
    assert rc == -1

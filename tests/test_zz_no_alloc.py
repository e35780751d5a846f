"""The allocation-free attention backward against the regular entry point.

Some callers cannot hand the library a scratch buffer because they cannot allocate at all at
that point (a capture in progress, an allocator they do not own).  ppu_attention_bwd_static
serves them from a fixed array inside the library.  Collected last on purpose: a failure here
must not hide the result of any other test in a run that stops at the first failure.
"""
import ctypes as C

import numpy as np
import pytest

pytestmark = pytest.mark.gpu


def _case(B, S, h, dh, seed):
    import torch
    g = torch.Generator(device="cpu").manual_seed(seed)
    d = h * dh
    qkv = torch.randn((B * S, 3 * d), generator=g).cuda().bfloat16()
    dU = torch.randn((B * S, d), generator=g).cuda().bfloat16()
    return qkv, dU


@pytest.mark.parametrize("backend,B,S,h,dh", [(0, 2, 333, 2, 64), (0, 1, 512, 4, 128), (1, 2, 64, 4, 16)])
def test_static_scratch_matches_regular_entry_point_twice(backend, B, S, h, dh):
    import torch
    from paper_2509_22418_b200 import ppu
    for call in range(2):                      # second call reuses the array the first one left
        qkv, dU = _case(B, S, h, dh, seed=100 * call + S)
        U, lse = ppu.ppu_attention_fwd(qkv, B, S, h, dh, backend=backend)
        ref = ppu.ppu_attention_bwd(qkv, U, lse, dU, B, S, h, dh, backend=backend)
        got = ppu.ppu_attention_bwd_static(qkv, U, lse, dU, B, S, h, dh, backend=backend)
        torch.cuda.synchronize()
        r, g = ref.float().cpu().numpy(), got.float().cpu().numpy()
        assert np.isfinite(g).all()
        assert np.abs(g - r).max() <= 2e-2 * np.abs(r).max()
        assert np.array_equal(g, r)            # same kernels, same order: identical bits


def test_static_scratch_rejects_sizes_beyond_its_limit():
    import torch
    from paper_2509_22418_b200 import ppu
    B, S, h, dh = 1, 64, 1, 64
    qkv, dU = _case(B, S, h, dh, seed=1)
    U, lse = ppu.ppu_attention_fwd(qkv, B, S, h, dh, backend=0)
    st = torch.cuda.current_stream().cuda_stream
    too_many = ppu.STATIC_SCRATCH_FLOATS // 64 + 1          # batch * 1 * 64 > limit
    rc = ppu.lib().ppu_attention_bwd_static(C.c_void_p(qkv.data_ptr()), C.c_void_p(U.data_ptr()),
                                            C.c_void_p(lse.data_ptr()), C.c_void_p(dU.data_ptr()),
                                            C.c_void_p(qkv.data_ptr()), too_many, 64, 1, 64, 0,
                                            C.c_void_p(st))
    assert rc == -2 and b"exceeds" in ppu.lib().ppu_last_error()


def test_static_scratch_against_the_oracle():
    """The same entry point against the CPU oracle's attention backward (Appendix C.1, MHA), so
    that this file stands on its own."""
    import torch
    from oracle import ppu_oracle as O
    from paper_2509_22418_b200 import ppu
    from tests.test_gpu_ops import _attention_case
    B, S, h, dh = 2, 200, 2, 64
    qkv, dU, L, U_ref, lse_ref, dU64 = _attention_case(B, S, h, dh, seed=77)
    U, lse = ppu.ppu_attention_fwd(qkv, B, S, h, dh, backend=0)
    dq, dk, dv = O._attention_bwd(O.Model(1, h * dh, h, 8, 8), L, dU64.reshape(B, S, h * dh), None)
    got = ppu.ppu_attention_bwd_static(qkv, U, lse, dU, B, S, h, dh, backend=0)
    torch.cuda.synchronize()
    g = got.float().cpu().numpy()
    d = h * dh
    for name, a, ref in (("dq", g[:, :d], dq), ("dk", g[:, d:2 * d], dk), ("dv", g[:, 2 * d:], dv)):
        ref = ref.reshape(B * S, d)
        assert np.abs(a - ref).max() <= 2e-2 * np.abs(ref).max(), name

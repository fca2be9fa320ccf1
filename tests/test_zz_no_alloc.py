"""The allocation-free attention entry point against the ordinary one.

tandem_decode_attention_static is for callers that cannot call cudaMalloc (host callbacks, processes whose
device memory belongs to a framework's pool, services that must not touch the allocator once they serve): its
work space (the per-row index arrays the kernel reads) is a buffer built into the library instead of a
caller-provided one.  It must give the same output as tandem_decode_attention, call after call, although every
call reuses that one buffer and finds the previous call's contents in it.  This file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import numpy as np
import pytest

from oracle import tandem_oracle as O
from paper_2402_08644_b200 import binding, build

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


def _inputs(B, H, dh, Td, To, seed):
    import torch
    g = torch.Generator().manual_seed(seed)
    mk = lambda *s: torch.randn(*s, generator=g).to(torch.bfloat16).cuda()
    return mk(B, H, dh), mk(B, H, Td, dh), mk(B, H, Td, dh), mk(B, H, To, dh), mk(B, H, To, dh)


def test_static_scratch_entry_point_matches_the_ordinary_one_twice_in_a_row():
    import torch
    build.build()
    binding.load_library()
    # two different shapes back to back: the second call meets the first call's contents in the buffer
    for B, H, dh, Td, To, seed in ((2, 16, 64, 1000, 4, 1), (3, 4, 128, 300, 2, 2)):
        q, kd, vd, ko, vo = _inputs(B, H, dh, Td, To, seed)
        want = binding.tandem_decode_attention(q, kd, vd, ko, vo)
        for call in range(2):
            out = torch.full_like(q, float("nan"))
            binding.tandem_decode_attention_static(q, kd, vd, ko, vo, out)
            torch.cuda.synchronize()
            diff = (out.float() - want.float()).abs().max().item()
            assert diff <= TOL_BF16, (B, H, dh, Td, To, call, diff)
            assert torch.equal(out, want)       # same kernels, same order: in fact bit-identical
        # and against the CPU checker directly, so that the two entry points cannot be wrong together
        f = lambda x: x.float().cpu().numpy().astype(np.float64)
        for b in range(B):
            for h in range(H):
                K = np.concatenate([f(kd[b, h]), f(ko[b, h])], 0)
                V = np.concatenate([f(vd[b, h]), f(vo[b, h])], 0)
                assert np.abs(f(out[b, h]) - O.attend(f(q[b, h]), K, V, 1)).max() < TOL_BF16


def test_static_scratch_entry_point_refuses_shapes_beyond_its_buffer():
    import torch
    build.build()
    lib = binding.load_library()
    B, H, dh, Td, To = 9000, 1, 32, 1, 0             # 8 bytes per sequence: more than the built-in 64 KiB
    assert lib.tandem_decode_attention_scratch_bytes(B, H, dh, Td, To) > binding.STATIC_SCRATCH_BYTES
    q = torch.zeros(B, H, dh, dtype=torch.bfloat16, device="cuda")
    kv = torch.zeros(1, dtype=torch.bfloat16, device="cuda")   # never read: the call must fail before any launch
    rc = lib.tandem_decode_attention_static(q.data_ptr(), kv.data_ptr(), kv.data_ptr(), kv.data_ptr(), kv.data_ptr(),
                                            q.data_ptr(), B, H, dh, Td, To, None)
    assert rc == 4
    assert b"built-in buffer" in lib.tandem_last_cuda_error()

"""The allocation-free decode-attention entry point (collected last on purpose).

pt_kernel_decode_attn_static serves callers that cannot obtain device memory at call time - a
serving loop that must stay away from the allocator once it is running, a host that owns no device
pool to carve scratch from.  It keeps its split plan and
partial results in an 8 MiB array built into the library, so all calls on a device share that
array and it still holds the previous call's data when the next one starts.  The test therefore
makes two different calls in a row and checks each against the ordinary entry point (which takes
a caller-owned scratch buffer), and checks that a problem too large for the array is refused."""
import numpy as np
import pytest

from tests.test_gpu_kernels import decode_case

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_matches_caller_scratch_entry_twice_in_a_row():
    import torch
    from paper_2602_07306_b200 import pt
    cases = [
        dict(T=2, B=3, nq=8, nkv=2, dh=128, ps=16, lens=[900, 33, 2047]),   # several key ranges per sequence
        dict(T=1, B=4, nq=4, nkv=4, dh=64, ps=16, lens=[5, 260, 1, 700]),   # different shape: stale plan and partials in the array
    ]
    for i, c in enumerate(cases):
        q, pool, bt, ref = decode_case(c["T"], c["B"], c["nq"], c["nkv"], c["dh"], c["ps"], c["lens"], seed=11 + i)
        want, st0 = pt.kernel_decode_attn(q, pool, bt, c["lens"], nq=c["nq"], nkv=c["nkv"], dh=c["dh"], ps=c["ps"])
        out = torch.empty_like(q)
        status = torch.zeros(16, dtype=torch.int32, device=q.device)
        got, st1 = pt.kernel_decode_attn_static(q, pool, bt, c["lens"], nq=c["nq"], nkv=c["nkv"], dh=c["dh"], ps=c["ps"],
                                                out=out, status=status)
        torch.cuda.synchronize()
        assert st0[:2].tolist() == [0, 0] and st1[:2].tolist() == [0, 0]
        g, w = got.float().cpu().numpy().astype(np.float64), want.float().cpu().numpy().astype(np.float64)
        d = np.abs(g - w)
        # same bounds as the kernel's own parity test; in practice the two entry points agree bit for bit
        assert d.max() <= 2e-2 * np.abs(w).max() and d.mean() <= 4e-3 * np.abs(w).mean(), f"call {i}: {d.max():.3e}"
        d = np.abs(g - ref)
        assert d.max() <= 2e-2 * np.abs(ref).max() and d.mean() <= 4e-3 * np.abs(ref).mean(), f"call {i} vs oracle: {d.max():.3e}"


def test_static_scratch_entry_refuses_oversized_problem():
    import torch
    from paper_2602_07306_b200 import pt
    q, pool, bt, _ = decode_case(1, 1, 2, 2, 64, 16, [20], seed=5)
    T, B, nq, dh = 8, 64, 8, 128                                   # needs about 34 MB of partials
    import ctypes as C
    n = C.c_size_t()
    pt.check(pt.lib().pt_kernel_decode_attn_scratch_bytes(T, B, nq, dh, C.byref(n)))
    assert n.value > (8 << 20)
    lens = (C.c_int32 * B)(*([16] * B))
    status = torch.zeros(16, dtype=torch.int32, device="cuda")
    rc = pt.lib().pt_kernel_decode_attn_static(q.data_ptr(), pool.data_ptr(), pool.stride(0), bt.data_ptr(), 1, lens,
                                               T, B, nq, nq, dh, 16, pool.shape[1], q.data_ptr(), status.data_ptr(), None)
    assert rc == 4 and b"built-in array" in pt.lib().pt_last_error()

"""Kernel-level parity through the C ABI: the tcgen05 track-grouped GEMM against the plain
definition sum_k a[t,m,k] w[t,n,k] evaluated in float64 from the same bf16-rounded operands."""
import numpy as np
import pytest

from paper_2602_07306_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _operands(T, M, N, K, seed):
    rng = np.random.default_rng(seed)
    a = I.round_to_bf16(rng.standard_normal((T, M, K), dtype=np.float32))
    w = I.round_to_bf16(rng.standard_normal((T, N, K), dtype=np.float32) * 0.05)
    return a, w


@pytest.mark.parametrize("T,M,N,K,bn,fold", [
    (1, 128, 128, 64, 128, False),        # one tile, one k-block
    (1, 128, 256, 256, 256, False),       # wide tile
    (2, 200, 384, 320, 128, False),       # ragged M, several tiles, tracks in the grid
    (3, 64, 2752, 128, 128, False),       # N tail (2752 = 21.5 x 128), M smaller than a tile
    (2, 300, 128, 1376, 128, False),      # K tail (1376 = 21.5 x 64)
    (4, 130, 512, 1376, 256, True),       # tracks folded into K (track-sync contraction)
    (2, 1024, 1024, 1024, 0, False),      # enough tiles for several per CTA, library-chosen width
])
def test_gemm_bf16_matches_definition(T, M, N, K, bn, fold):
    import torch
    from paper_2602_07306_b200 import pt
    a, w = _operands(T, M, N, K, seed=M + N + K)
    ref = np.einsum("tmk,tnk->tmn", a.astype(np.float64), w.astype(np.float64))
    if fold:
        ref = ref.sum(0, keepdims=True)
    da = torch.from_numpy(a).cuda().to(torch.bfloat16)
    dw = torch.from_numpy(w).cuda().to(torch.bfloat16)
    c, status = pt.kernel_gemm_bf16(da, dw, bn=bn, fold_tracks=fold)
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    got = c.cpu().numpy().astype(np.float64)
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err <= 2e-6 * np.sqrt(K * (T if fold else 1)), f"max-rel {err:.3e}"     # fp32 accumulation of exact bf16 products

"""How accurate can a bf16 PT forward be at the width of the T=8 model?

The oracle computes in float64 from bf16-rounded weights and inputs and rounds nothing else.  Any
implementation that feeds bf16 tensor-core operands must round at least the operands of its
contractions (the gain-scaled stream in front of the QKV and gate/up projections, q, the
probabilities, the attention output, the SwiGLU output) and the cached K and V.  This test applies
exactly those roundings, and nothing else, inside the oracle's own arithmetic for the first track
block of the T=8, hidden-1024 model (the error settles there: later blocks start from the sum of the
tracks, which carries it on unchanged) and measures the mean relative error of the stream against the
unrounded run.  It comes out above the 2e-3 target, which is why the full-size GPU tests use
helpers.DEEP_MEAN_TOL; the small workloads, whose deltas are smaller than their stream, stay below
2e-3 and are held to it."""
import numpy as np

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp


def _layer(h, w, pos, nq, nkv, dh, rnd):
    R = (lambda a: I.round_to_bf16(np.asarray(a, np.float32)).astype(np.float64)) if rnd else (lambda a: a)
    S = h.shape[0]
    rinv = 1.0 / np.sqrt(np.mean(h * h, -1, keepdims=True) + 1e-6)
    a = R(h * w["g1"]) * rinv
    q = R(O.rope((a @ w["wq"].T).reshape(S, nq, dh), pos, 1e4))
    k = R(O.rope((a @ w["wk"].T).reshape(S, nkv, dh), pos, 1e4))
    v = R((a @ w["wv"].T).reshape(S, nkv, dh))
    o = np.empty_like(q)
    for i in range(nq):
        j = i // (nq // nkv)
        s = q[:, i] @ k[:, j].T / np.sqrt(dh)
        s = np.where(pos[None, :] <= pos[:, None], s, -np.inf)
        p = np.exp(s - s.max(-1, keepdims=True))
        o[:, i] = (R(p) @ v[:, j]) / p.sum(-1, keepdims=True)
    h = h + R(o.reshape(S, -1)) @ w["wo"].T
    rinv = 1.0 / np.sqrt(np.mean(h * h, -1, keepdims=True) + 1e-6)
    c = R(h * w["g2"]) * rinv
    return h + R(O.silu(c @ w["wg"].T) * (c @ w["wu"].T)) @ w["wd"].T


import pytest


@pytest.mark.parametrize("T,D,H,nq,nkv,F,tol", [(8, 8, 1024, 8, 8, 2816, Hp.DEEP_MEAN_TOL), (4, 2, 2048, 16, 4, 5632, Hp.WIDE_MEAN_TOL)])
def test_rounding_only_the_tensor_core_operands_already_exceeds_2e_3_on_the_wide_models(T, D, H, nq, nkv, F, tol):
    S = 12
    wl = I.Workload("block", T=T, L=D, D=D, hidden=H, heads=nq, kv_heads=nkv, ffn=F, dtype="bf16",
                    mode="prefill", batch=1, seq=S)
    ws = I.WeightSource(wl)
    x = I.prefill_inputs(wl).astype(np.float64)
    pos = np.arange(S)
    exact = [x[t, 0].copy() for t in range(T)]
    rounded = [x[t, 0].copy() for t in range(T)]
    for l in range(D):
        for t in range(T):
            w = {k: np.asarray(v, np.float64) for k, v in ws.get(t, l).items()}
            exact[t] = _layer(exact[t], w, pos, nq, nkv, wl.head_dim, False)
            rounded[t] = _layer(rounded[t], w, pos, nq, nkv, wl.head_dim, True)
    e, r = sum(exact), sum(rounded)                           # the track-sync that closes the block
    mx, mean = Hp.rel_errs(r, e)
    print(f"hidden {H}: floor mean-rel {mean:.3e}, max-rel {mx:.3e}")
    assert 2.0e-3 < mean < tol, mean
    assert mx < 2e-2

"""The workspace-free TL entry point against the regular one.

bitnet_mpgemv_tl_noalloc serves callers that cannot allocate device memory (frozen or fully committed
allocator, latency-critical loops, plug-ins that only get input and output buffers): its split-K
scratch is a fixed array inside the library.  It must give exactly what bitnet_mpgemm gives with a
caller-owned workspace, call after call, although every call reuses the same array.  This file is
collected last so that a run stopping at the first failure has already run everything else.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth

pytestmark = pytest.mark.gpu

REL_TOL = 1e-6


def _case(fmt, M, K, T, seed, want_inputs=False):
    w = synth.ternary(seed, 1, M, K, 1 / 3, 1 / 3)
    x = synth.normal(seed, 2, T, K)
    q, sc, _ = bn.bitnet_quant_act(x.cuda())
    blob = bn.pack(fmt, w.cuda())
    return (blob, q, sc, w, x) if want_inputs else (blob, q, sc)


@pytest.mark.parametrize("fmt,M,K,T", [("tl2", 64, 28672, 1), ("tl2", 96, 8192, 2), ("tl1", 32, 14336, 3),
                                       ("tl2", 32, 96, 1)])
def test_noalloc_matches_workspace_entry_point_twice(fmt, M, K, T):
    w_scale = 0.625
    for call in range(2):                      # two calls in a row share the built-in scratch
        blob, q, sc, w, x = _case(fmt, M, K, T, seed=40 + call, want_inputs=True)
        y_ref, acc_ref = bn.bitnet_mpgemm(fmt, blob, w_scale, M, K, q, sc, want_acc=True)
        y = torch.full((T, M), float("nan"), dtype=torch.float32, device="cuda")
        acc = torch.full((T, M), -7, dtype=torch.int32, device="cuda")
        bn.bitnet_mpgemv_tl_noalloc(fmt, blob, w_scale, M, K, q, sc, y, acc)
        torch.cuda.synchronize()
        assert torch.equal(acc, acc_ref)
        yr = y_ref.double().cpu().numpy()
        err = np.abs(y.double().cpu().numpy() - yr)
        assert np.all(err <= REL_TOL * np.abs(yr))
        # and directly against the CPU oracle
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(acc.cpu().numpy(), acc_ref)
        y_or = oracle.dequant(acc_ref, sc_ref, w_scale)
        assert np.all(np.abs(y.double().cpu().numpy() - y_or) <= REL_TOL * np.abs(y_or))


def test_noalloc_rejects_sizes_beyond_its_scratch():
    blob, q, sc = _case("tl2", 32, 96, 1, seed=44)
    y = torch.empty((1, 32), dtype=torch.float32, device="cuda")
    with pytest.raises(bn.BitnetError, match="workspace"):
        bn.bitnet_mpgemv_tl_noalloc("tl2", blob, 1.0, bn.NOALLOC_MAX_M + 32, 96, q, sc, y)
    with pytest.raises(bn.BitnetError, match="workspace"):
        bn.bitnet_mpgemv_tl_noalloc("tl2", blob, 1.0, 32, bn.NOALLOC_MAX_K + 96, q, sc, y)
    q9 = torch.zeros((9, 96), dtype=torch.int8, device="cuda")
    sc9 = torch.ones(9, dtype=torch.float32, device="cuda")
    y9 = torch.empty((9, 32), dtype=torch.float32, device="cuda")
    with pytest.raises(bn.BitnetError, match="workspace"):
        bn.bitnet_mpgemv_tl_noalloc("tl2", blob, 1.0, 32, 96, q9, sc9, y9)
    with pytest.raises(bn.BitnetError, match="invalid"):
        bn.bitnet_mpgemv_tl_noalloc("i2s", blob, 1.0, 32, 96, q, sc, y)

"""Seeded random shapes through the list calls against the oracle: every format at 1..8 tokens, I2_S up to 128, ragged row and column
counts, short and long rows, lists that mix formats and shapes in one call.  The shapes are drawn so that each case
stays small enough for the oracle to finish in well under a second."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth
from helpers import Guarded, check_y, npy
from test_gpu_group import Item, run_group

pytestmark = pytest.mark.gpu


def _draw_shape(rng, fmt):
    T = int(rng.integers(1, 9))
    if fmt == "i2s":
        M = int(rng.integers(1, 400))
        K = 64 * int(rng.integers(1, 200))
    else:
        M = 32 * int(rng.integers(1, 12))
        K = int(rng.choice([2, 4])) * int(rng.integers(1, 3000))      # even, often not a multiple of 4, 64 or 96
    if rng.random() < 0.15:
        K = (28672 if fmt == "i2s" else 28672 + 2 * int(rng.integers(0, 3)))
        M = min(M, 96) if fmt == "i2s" else 32
    return M, K, T


@pytest.mark.parametrize("seed", range(6))
def test_random_lists_of_every_format(seed):
    rng = np.random.default_rng(1000 + seed)
    items = []
    for i in range(10):
        fmt = str(rng.choice(["i2s", "tl1", "tl2"]))
        M, K, T = _draw_shape(rng, fmt)
        items.append(Item(fmt, M, K, T, 5000 + 100 * seed + i, w_scale=float(rng.choice([0.5, 0.625, 1.0]))))
    run_group(items)
    for it in items:
        it.check()


@pytest.mark.parametrize("seed", range(4))
def test_random_lists_beyond_ternary(seed):
    rng = np.random.default_rng(2000 + seed)
    descs, keep = [], []
    for i in range(8):
        C = int(rng.choice([3, 4, 5]))
        T = int(rng.integers(1, 9))
        M = 32 * int(rng.integers(1, 12))
        K = 4 * int(rng.integers(48, 2500))                 # a multiple of 4, at least three tiles
        if rng.random() < 0.15:
            M, K = 32, 28672 + 4 * int(rng.integers(0, 3))
        w = synth.uniform_alphabet(6000 + seed, i, M, K, C)
        x = synth.normal(6000 + seed, 100 + i, T, K)
        gq, gsc = Guarded((T, K), torch.int8), Guarded((T,), torch.float32)
        gy, gacc = Guarded((T, M), torch.float32), Guarded((T, M), torch.int32)
        descs.append(dict(C=C, g=2, packed=bn.bitnet_pack_elut(C, 2, w.cuda()), w_scale=0.75, M=M, K=K, x=x.cuda(),
                          q=gq.t, act_scale=gsc.t, y=gy.t, acc_out=gacc.t))
        keep.append((w, x, (gq, gsc, gy, gacc)))
    bn.bitnet_elut_linear_group(bn.make_elut_group(descs))
    torch.cuda.synchronize()
    assert bn.bitnet_device_status() == 0
    for d, (w, x, guards) in zip(descs, keep):
        for g in guards:
            assert g.intact(), (d["C"], d["M"], d["K"])
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(d["q"]), q_ref)
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(d["acc_out"]), acc_ref), (d["C"], d["M"], d["K"], x.shape[0])
        check_y(d["y"], acc_ref, sc_ref, 0.75)


@pytest.mark.parametrize("seed", range(5))
def test_random_i2s_lists_from_nine_to_128_tokens(seed):
    """I2_S lists whose items have 1 to 128 tokens in random order: neighbouring items change between the grouped
    kernel's one- and two-group forms, the streaming tensor-core kernel's 64- and 128-token tiles and the single-call
    kernels (rows shorter than 2048 columns), ragged row counts, K with odd numbers of 256-column chunks."""
    rng = np.random.default_rng(3000 + seed)
    items = []
    for i in range(12):
        T = int(rng.choice([int(rng.integers(1, 9)), int(rng.integers(9, 17)), int(rng.integers(17, 65)),
                            int(rng.integers(65, 129))]))
        M = int(rng.integers(1, 300))
        K = 64 * int(rng.integers(8, 130))
        if rng.random() < 0.12:
            M, K = int(rng.integers(1, 64)), 28672
        items.append(Item("i2s", M, K, T, 7000 + 100 * seed + i, w_scale=float(rng.choice([0.5, 0.625, 1.0]))))
    run_group(items)
    for it in items:
        it.check()

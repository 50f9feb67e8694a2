"""Element-wise tables beyond ternary (App. A; Table 3) on the GPU against the CPU oracle: pair indices of weights of
cardinality C = 3, 4, 5 -- packer bytes, round trip, and the grouped decode kernel (1..8 tokens) element by element.
"""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth
from helpers import Guarded, check_y, npy

pytestmark = pytest.mark.gpu


def _weights(C, M, K, seed=11, tid=1):
    return synth.uniform_alphabet(seed, tid, M, K, C)


@pytest.mark.parametrize("C", [3, 4, 5])
@pytest.mark.parametrize("M,K", [(32, 64), (64, 130), (96, 4096), (32, 2)])
def test_pack_elut_bytes_and_round_trip(C, M, K):
    w = _weights(C, M, K)
    blob = bn.bitnet_pack_elut(C, 2, w.cuda())
    ref = oracle.pack_elut2(C, w.numpy())
    assert blob.numel() == ref.size == bn.bitnet_elut_packed_bytes(C, 2, M, K)
    assert np.array_equal(npy(blob), ref)
    assert torch.equal(bn.bitnet_unpack_elut(C, 2, blob, M, K).cpu(), w)


def test_pack_elut_rejects_values_outside_the_alphabet_and_unbuilt_forms():
    for C in (3, 4, 5):
        w = torch.zeros((32, 64), dtype=torch.int8)
        w[3, 7] = -(C // 2) + C
        with pytest.raises(bn.BitnetError, match="alphabet"):
            bn.bitnet_pack_elut(C, 2, w.cuda())
    assert bn.bitnet_elut_packed_bytes(5, 3, 32, 96) == 0 and bn.bitnet_elut_packed_bytes(6, 2, 32, 64) == 0
    assert bn.bitnet_elut_packed_bytes(5, 2, 33, 64) == 0 and bn.bitnet_elut_packed_bytes(5, 2, 32, 65) == 0
    assert bn.bitnet_elut_packed_bytes(5, 2, 64, 128) * 8 == 5 * 64 * 128 // 2      # 2.5 bits per weight
    assert bn.bitnet_elut_packed_bytes(4, 2, 64, 128) * 8 == 4 * 64 * 128 // 2      # 2 bits per weight


def _run(items_spec, fused):
    """items_spec: list of (C, M, K, T, seed).  Runs one bitnet_elut_linear_group call; returns per item the device
    results and the host inputs."""
    items, keep = [], []
    for C, M, K, T, seed in items_spec:
        w = _weights(C, M, K, seed, 1)
        x = synth.normal(seed, 2, T, K)
        blob = bn.bitnet_pack_elut(C, 2, w.cuda())
        gq, gsc = Guarded((T, K), torch.int8), Guarded((T,), torch.float32)
        gy, gacc = Guarded((T, M), torch.float32), Guarded((T, M), torch.int32)
        d = dict(C=C, g=2, packed=blob, w_scale=0.375 + 0.125 * C, M=M, K=K, q=gq.t, act_scale=gsc.t, y=gy.t, acc_out=gacc.t)
        if fused:
            d["x"] = x.cuda()
        else:
            q, sc, _ = bn.bitnet_quant_act(x.cuda())
            gq.t.copy_(q)
            gsc.t.copy_(sc)
        items.append(d)
        keep.append((w, x, (gq, gsc, gy, gacc)))
    bn.bitnet_elut_linear_group(bn.make_elut_group(items))
    torch.cuda.synchronize()
    return items, keep


def _check(items, keep):
    for d, (w, x, guards) in zip(items, keep):
        for gd in guards:
            assert gd.intact(), (d["C"], d["M"], d["K"])
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(d["q"]), q_ref)
        assert np.array_equal(npy(d["act_scale"]).view(np.uint32), sc_ref.view(np.uint32))
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(d["acc_out"]), acc_ref), (d["C"], d["M"], d["K"])
        check_y(d["y"], acc_ref, sc_ref, d["w_scale"])


@pytest.mark.parametrize("C", [3, 4, 5])
@pytest.mark.parametrize("fused", [False, True])
def test_elut_decode_single_linears(C, fused):
    # several tiles and a ragged last tile (K % 64 != 0), few and many row blocks, 1..8 tokens
    for M, K, T in [(32, 192, 1), (64, 1028, 1), (96, 4096, 3), (2048, 4100, 1), (160, 8192, 8), (64, 28672, 2)]:
        _check(*_run([(C, M, K, T, 20 + T)], fused))


def test_elut_decode_agrees_with_the_lookup_form_of_the_oracle():
    # the packed blob read back by the oracle's table-setup + lookup accumulation (App. A, "ELUT mpGEMM")
    for C in (4, 5):
        M, K, T = 64, 1024, 2
        items, keep = _run([(C, M, K, T, 5)], True)
        w, x, _ = keep[0]
        q_ref, _, _ = oracle.quant_act(x.numpy())
        acc_lut = oracle.elut2_mpgemm(C, npy(items[0]["packed"]), M, K, q_ref)
        assert np.array_equal(npy(items[0]["acc_out"]), acc_lut)


def test_elut_group_of_mixed_cardinalities_and_shapes():
    spec = [(5, 64, 4096, 1, 1), (5, 4096, 1024, 1, 2), (5, 32, 14336, 4, 3), (4, 96, 4096, 1, 4), (4, 1024, 2048, 2, 5),
            (3, 64, 8192, 1, 6), (5, 128, 8192, 8, 7)]
    _check(*_run(spec, True))
    _check(*_run(spec, False))


def test_elut_long_rows_in_parts_and_full_width_layer():
    # 8 tokens x 28672 columns do not fit beside the decode table: the row is walked in parts
    _check(*_run([(5, 64, 28672, 8, 9), (4, 32, 28672, 7, 10)], True))
    # a 100B-shaped gate/up projection at C = 5 (sampled rows of the oracle would do; 1792 row blocks run whole here)
    C, M, K, T = 5, 57344, 8192, 1
    w = synth.uniform_alphabet(3, 1, M, K, C, device="cuda")
    x = synth.normal(3, 2, T, K)
    blob = bn.bitnet_pack_elut(C, 2, w)
    q = torch.empty((T, K), dtype=torch.int8, device="cuda")
    sc = torch.empty(T, dtype=torch.float32, device="cuda")
    y = torch.empty((T, M), dtype=torch.float32, device="cuda")
    acc = torch.empty((T, M), dtype=torch.int32, device="cuda")
    bn.bitnet_elut_linear_group(bn.make_elut_group([dict(C=C, g=2, packed=blob, w_scale=1.0, M=M, K=K, x=x.cuda(), q=q,
                                                         act_scale=sc, y=y, acc_out=acc)]))
    torch.cuda.synchronize()
    q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
    rows = np.unique(np.concatenate([np.arange(0, 64), np.arange(M - 64, M), np.random.default_rng(1).integers(0, M, 512)]))
    acc_ref = oracle.mpgemm_def(q_ref, w[torch.as_tensor(rows).cuda()].cpu().numpy())
    assert np.array_equal(npy(acc)[:, rows], acc_ref)
    check_y(y[:, torch.as_tensor(rows).cuda()], acc_ref, sc_ref, 1.0)


def test_elut_malformed_items_are_refused():
    C, M, K = 5, 32, 256
    blob = bn.bitnet_pack_elut(C, 2, _weights(C, M, K).cuda())
    q = torch.zeros((1, K), dtype=torch.int8, device="cuda")
    sc = torch.ones(1, dtype=torch.float32, device="cuda")
    y = torch.zeros((1, M), dtype=torch.float32, device="cuda")
    base = dict(C=C, g=2, packed=blob, w_scale=1.0, M=M, K=K, q=q, act_scale=sc, y=y)
    with pytest.raises(bn.BitnetError, match="unsupported"):
        bn.bitnet_elut_linear_group(bn.make_elut_group([dict(base, g=3)]))
    with pytest.raises(bn.BitnetError, match="unsupported"):
        bn.bitnet_elut_linear_group(bn.make_elut_group([dict(base, C=7)]))
    with pytest.raises(bn.BitnetError, match="unsupported"):
        bn.bitnet_elut_linear_group(bn.make_elut_group([dict(base, K=66)]))       # K % 4 != 0
    q9 = torch.zeros((9, K), dtype=torch.int8, device="cuda")
    with pytest.raises(bn.BitnetError, match="invalid"):
        bn.bitnet_elut_linear_group(bn.make_elut_group([dict(base, q=q9)]))       # more than 8 tokens
    bn.bitnet_elut_linear_group(bn.make_elut_group([]))                           # an empty list is fine


def test_cardinality4_through_the_decode_table_in_a_child_process():
    """Cardinality 4 is decoded by masks by default (its pair index is two 2-bit codes); BITNET_ELUT4=table, read once
    per process, sends it through the decode table like cardinality 3 and 5.  Same integers either way."""
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import sys; sys.path.insert(0, 'tests')\n"
            "from test_gpu_elut import _run, _check\n"
            "for fused in (False, True):\n"
            "    for M, K, T in [(32, 192, 1), (64, 1028, 1), (96, 4096, 3), (2048, 4100, 1), (160, 8192, 8), (64, 28672, 2)]:\n"
            "        _check(*_run([(4, M, K, T, 20 + T)], fused))\n"
            "print('ok')\n")
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, BITNET_ELUT4="table"),
                         capture_output=True, text=True, timeout=900)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr[-2000:]

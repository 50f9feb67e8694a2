"""The C-ABI library loads without a GPU and exports every symbol the header declares; host-side
argument validation returns status codes without launching anything."""
import ctypes as C
import os
import re

import pytest

import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import build as bn_build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    bn_build.build()
    return bn.lib()


def header_symbols():
    text = open(os.path.join(ROOT, "include", "bitnet_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bitnet_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    names = header_symbols()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert set(bn.SYMBOLS) <= set(names)


def test_status_strings(L):
    assert bn.status_string(0) == "ok"
    for rc in range(1, 7):
        assert bn.status_string(rc) not in ("ok", "unknown status")
    assert bn.status_string(99) == "unknown status"


def test_size_queries(L):
    assert bn.bitnet_i2s_packed_bytes(1536, 1536) == 1536 * 1536 // 4
    assert bn.bitnet_i2s_packed_bytes(3200, 8640) == 3200 * 8704 // 4
    assert bn.bitnet_i2s_packed_bytes(3, 64) == 1024
    assert bn.bitnet_i2s_packed_bytes(16, 100) == 0                      # K % 64 != 0
    assert bn.bitnet_tl_packed_bytes("tl2", 32, 8192) == 85 * 640 + 512
    assert bn.bitnet_tl_packed_bytes("tl1", 64, 130) == 2 * 3 * 512
    assert bn.bitnet_tl_packed_bytes("tl2", 33, 96) == 0
    assert bn.bitnet_tl_packed_bytes("tl2", 32, 96, 100) == 0            # bk3 not a multiple of 96
    assert bn.bitnet_tl_num_groups("tl2", 8192) == 86 * 32
    assert bn.bitnet_mpgemm_workspace_bytes("i2s", 1, 8192, 8192) == 0
    assert bn.bitnet_mpgemm_workspace_bytes("i2s", 1, 8192, 28672) == 0        # in-CTA reduction
    assert bn.bitnet_mpgemm_workspace_bytes("i2s", 3, 1 << 20, 8192) == 0       # small decode batches: none
    # batches whose codes crowd the decode kernel, and 9 to 64 tokens: the T x M sums of the K-slices
    assert 0 <= bn.bitnet_mpgemm_workspace_bytes("i2s", 8, 1 << 20, 1 << 17) - 8 * (1 << 20) * 4 <= 4096
    assert 0 <= bn.bitnet_mpgemm_workspace_bytes("i2s", 33, 8192, 28672) - 33 * 8192 * 4 <= 4096
    # prefill kernel: none when the output tiles fill the SMs, the T x M sums when K is cut to fill them
    assert bn.bitnet_mpgemm_workspace_bytes("i2s", 2048, 14336, 4096) == 0
    assert bn.bitnet_mpgemm_workspace_bytes("i2s", 65, 57344, 8192) == 0
    assert bn.bitnet_mpgemm_workspace_bytes("i2s", 65, 8192, 28672) == 65 * 8192 * 4
    assert bn.bitnet_mpgemm_workspace_bytes("tl2", 1, 8192, 28672) >= 2 * 8192 * 4


def test_host_validation_returns_codes_without_a_gpu(L):
    null = C.c_void_p(None)
    fake = C.c_void_p(4096)          # never dereferenced: validation fails first
    odd = C.c_void_p(4100)
    assert L.bitnet_quant_act(null, 1, 64, 0, fake, fake, null, null) == 1
    assert L.bitnet_quant_act(fake, 0, 64, 0, fake, fake, null, null) == 1
    assert L.bitnet_quant_act(odd, 1, 64, 0, fake, fake, null, null) == 1
    assert L.bitnet_pack_i2s(fake, 8, 100, fake, 1 << 20, null, null) == 2
    assert L.bitnet_pack_i2s(fake, 8, 128, fake, 16, null, null) == 1      # blob too small
    assert L.bitnet_pack_tl(0, fake, 32, 96, 0, fake, 1 << 20, null, null) == 1   # I2_S is not a TL format
    assert L.bitnet_pack_tl(2, fake, 48, 96, 0, fake, 1 << 20, null, null) == 2   # M % 32
    assert L.bitnet_pack_tl(2, fake, 32, 95, 0, fake, 1 << 20, null, null) == 2   # K odd
    assert L.bitnet_mpgemm(0, fake, 1.0, 64, 100, 0, fake, fake, 1, fake, null, null, 0, null) == 2
    assert L.bitnet_mpgemm(0, fake, 1.0, 64, 128, 0, fake, fake, 0, fake, null, null, 0, null) == 1
    assert L.bitnet_mpgemm(0, fake, 1.0, 64, 128, 0, odd, fake, 1, fake, null, null, 0, null) == 1
    # lookup-table kernel (rows the scan kernel does not take: K not a multiple of 4) without the workspace it keeps
    # its tables in
    assert L.bitnet_mpgemm(1, fake, 1.0, 64, 28674, 0, fake, fake, 1, fake, null, null, 0, null) == 3
    # element-wise tables beyond ternary: only pairs of cardinality 3, 4, 5 are built
    assert L.bitnet_elut_packed_bytes(5, 2, 64, 128) == 64 * 128 * 5 // 16
    assert L.bitnet_elut_packed_bytes(5, 3, 64, 126) == 0 and L.bitnet_elut_packed_bytes(6, 2, 64, 128) == 0
    assert L.bitnet_pack_elut(5, 3, fake, 32, 96, fake, 1 << 20, null, null) == 2
    assert L.bitnet_pack_elut(5, 2, fake, 48, 96, fake, 1 << 20, null, null) == 2   # M % 32
    assert L.bitnet_pack_elut(5, 2, null, 32, 96, fake, 1 << 20, null, null) == 1
    assert L.bitnet_pack_elut(5, 2, fake, 32, 128, fake, 16, null, null) == 1       # blob too small
    assert L.bitnet_elut_linear_group(null, 1, null) == 1 and L.bitnet_elut_linear_group(null, 0, null) == 0
    # bitnet_linear validates the shape before it plans a launch (K = 0 or negative must not reach a division)
    for T in (1, 6, 8):
        assert L.bitnet_linear(0, fake, 1.0, 64, 0, 0, fake, T, fake, fake, fake, null, fake, 1 << 20, null) == 1
        assert L.bitnet_linear(0, fake, 1.0, 64, -16, 0, fake, T, fake, fake, fake, null, fake, 1 << 20, null) == 1
    # the grouped call rejects a malformed list before anything is queued
    assert L.bitnet_linear_group(null, 1, null) == 1
    assert L.bitnet_linear_group(null, 0, null) == 0
    assert L.bitnet_mpgemm(1, fake, 1.0, 32, 64, 0, fake, fake, 1, fake, null, fake, 16, null) == 3   # too small


def test_missing_library_raises(monkeypatch, tmp_path):
    monkeypatch.setattr(bn, "_lib", None)
    monkeypatch.setattr(bn, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(bn.BitnetError):
        bn.lib()

"""Pins of the CPU oracle against things other than itself.

Each test checks the oracle against a fact fixed by the paper or by mathematics: printed table rows
(golden text fixtures), closed forms, brute force written independently in numpy / pure Python,
invariants, and cross-format equality (the paper's "lossless" claim for I2_S, TL1_1 and TL2_1).
"""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLD = os.path.join(os.path.dirname(__file__), "golden")
rng = np.random.default_rng(1234)


def rand_ternary(M, K, p0=1 / 3):
    u = rng.random((M, K))
    return np.where(u < p0, 0, np.where(u < p0 + (1 - p0) / 2, 1, -1)).astype(np.int8)


def rand_q(T, K):
    return rng.integers(-127, 128, size=(T, K)).astype(np.int8)


# ----------------------------------------------------------------------------- quantiser (Alg. 1 Phase 1)
def test_quant_half_even_closed_form():
    # amax = 127 makes the multiplier exactly 1, so q = rint(x) with ties to even
    x = np.array([[127.0, 0.5, 1.5, 2.5, -0.5, -1.5, 126.5, -2.5, 3.5]], np.float32)
    q, sc, sm = oracle.quant_act(x)
    assert q.tolist() == [[127, 0, 2, 2, 0, -2, 126, -2, 4]]
    assert sc[0] == np.float32(1.0)
    assert sm[0] == sum(q[0].tolist())


def test_quant_extreme_maps_to_127_and_scale():
    x = rng.standard_normal((5, 333)).astype(np.float32)
    q, sc, sm = oracle.quant_act(x)
    for t in range(5):
        k = np.argmax(np.abs(x[t]))
        assert abs(int(q[t, k])) == 127
        assert np.sign(q[t, k]) == np.sign(x[t, k])
        assert sc[t] == np.float32(np.abs(x[t]).max()) / np.float32(127.0)
        assert q[t].min() >= -127
        assert sm[t] == q[t].astype(np.int64).sum()


def test_quant_power_of_two_invariance_and_odd_symmetry():
    x = rng.standard_normal((3, 257)).astype(np.float32)
    q0, s0, _ = oracle.quant_act(x)
    for j in (-7, 3, 11):
        qj, sj, _ = oracle.quant_act(x * np.float32(2.0 ** j))
        assert np.array_equal(qj, q0)
        assert np.array_equal(sj, s0 * np.float32(2.0 ** j))
    qn, sn, smn = oracle.quant_act(-x)
    assert np.array_equal(qn, -q0) and np.array_equal(sn, s0)


def test_quant_matches_float64_rounding_away_from_ties():
    # independent evaluation in float64: wherever x*s is further than 1e-3 from a .5 tie the rounded
    # integer is unambiguous and must agree
    x = rng.standard_normal((4, 1000)).astype(np.float32)
    q, sc, _ = oracle.quant_act(x)
    for t in range(4):
        amax = np.abs(x[t]).astype(np.float64).max()
        p = x[t].astype(np.float64) * 127.0 / amax
        clear = np.abs(p - np.floor(p) - 0.5) > 1e-3
        assert np.array_equal(q[t][clear], np.rint(p[clear]).astype(np.int8))


def test_quant_zero_row_and_per_tensor():
    x = np.zeros((2, 64), np.float32)
    x[1, 3] = 2.0
    q, sc, sm = oracle.quant_act(x)
    assert not q[0].any() and sc[0] == np.float32(1e-5) / np.float32(127.0) and sm[0] == 0
    assert q[1, 3] == 127
    qt, sct, _ = oracle.quant_act(x, per_tensor=True)
    assert sct[0] == sct[1] == np.float32(2.0) / np.float32(127.0)
    x2 = rng.standard_normal((3, 100)).astype(np.float32)
    qa, sa, _ = oracle.quant_act(x2, per_tensor=True)
    qb, sb, _ = oracle.quant_act(x2.reshape(1, -1))
    assert np.array_equal(qa.reshape(-1), qb.reshape(-1)) and np.all(sa == sb[0])


def test_quant_outlier_recipe_range():
    # two +-20 outliers among N(0,1) values: amax = 20 so a value |x| <= 6.3 quantises to |q| <= 40
    x = rng.standard_normal((1, 1536)).astype(np.float32).clip(-6.2, 6.2)
    x[0, 10], x[0, 900] = 20.0, -20.0
    q, sc, _ = oracle.quant_act(x)
    assert q[0, 10] == 127 and q[0, 900] == -127
    mask = np.ones(1536, bool)
    mask[[10, 900]] = False
    assert np.abs(q[0][mask]).max() <= 40


# ----------------------------------------------------------------------------- definition (Alg. 1 Phase 2, Eq. 1)
def test_definition_brute_force_all_rows_tiny():
    K = 5
    rows = np.array(list(itertools.product((-1, 0, 1), repeat=K)), np.int8)  # all 3^5 weight rows
    q = np.array([[1, -2, 3, -4, 5], [127, -128, 127, -128, 0], [0, 0, 0, 0, 0]], np.int8)
    acc = oracle.mpgemm_def(q, rows)
    for t in range(q.shape[0]):
        for m in range(rows.shape[0]):
            s = 0
            for k in range(K):
                s += int(q[t][k]) * int(rows[m][k])
            assert acc[t, m] == s


def test_definition_vs_numpy_matmul_and_not_transposed():
    T, M, K = 3, 37, 129
    q, w = rand_q(T, K), rand_ternary(M, K)
    acc = oracle.mpgemm_def(q, w)
    assert acc.shape == (T, M)
    assert np.array_equal(acc, q.astype(np.int64) @ w.astype(np.int64).T)


def test_definition_permutation_and_linearity():
    T, M, K = 2, 16, 96
    q, w = rand_q(T, K), rand_ternary(M, K)
    perm = rng.permutation(K)
    assert np.array_equal(oracle.mpgemm_def(q, w), oracle.mpgemm_def(q[:, perm], w[:, perm]))
    wa, wb = w.copy(), w.copy()
    wa[:, K // 2:] = 0
    wb[:, :K // 2] = 0
    assert np.array_equal(oracle.mpgemm_def(q, w), oracle.mpgemm_def(q, wa) + oracle.mpgemm_def(q, wb))


def test_dequant_closed_form():
    acc = np.array([[3, -5, 0]], np.int32)
    y = oracle.dequant(acc, np.array([0.5], np.float32), 0.25)
    assert y.tolist() == [[0.375, -0.625, 0.0]]


# ----------------------------------------------------------------------------- I2_S packing (Table 1: 2 bpw)
def test_i2s_size_and_bpw():
    assert oracle.i2s_packed_bytes(1536, 1536) == 1536 * 1536 // 4        # exactly 2 bits per weight
    assert oracle.i2s_packed_bytes(3200, 8640) == 3200 * 8704 // 4        # K padded to 256 columns
    assert oracle.i2s_packed_bytes(8192, 28672) * 8 == 2 * 8192 * 28672
    assert oracle.i2s_packed_bytes(3, 64) == 16 * 256 // 4                # rows padded to 16


def test_i2s_round_trip_and_padding_code():
    for (M, K) in [(3, 128), (5, 192), (7, 64), (2, 8640 // 8), (17, 512), (8, 256)]:
        w = rand_ternary(M, K)
        p = oracle.pack_i2s(w)
        assert p.size == oracle.i2s_packed_bytes(M, K)
        assert np.array_equal(oracle.unpack_i2s(p, M, K), w)
    # all-zero weights: every 2-bit field, padding included, holds code 1
    p = oracle.pack_i2s(np.zeros((3, 64), np.int8))
    assert p.size == 1024 and np.all(p == 0b01010101)


def _i2s_byte_and_shift(m, k, K):
    """The documented position of weight (m, k), written out independently of the oracle."""
    kp = -(-K // 256) * 256
    rb, r, c, kk = m // 16, m % 16, k // 256, k % 256
    word = 2 * (kk // 32) + (kk % 8) // 4
    return rb * 4 * kp + c * 1024 + r * 64 + 4 * word + kk % 4, 2 * ((kk % 32) // 8)


def test_i2s_documented_bit_positions():
    # every column of one chunk plus positions in other rows, row blocks and chunks; checked against
    # hand-built bytes
    M, K = 19, 512
    probes = [(0, k) for k in range(256)] + [(3, 5), (7, 255), (8, 0), (10, 300), (15, 511), (1, 256), (16, 0), (18, 77)]
    for (m, k) in probes:
        for val in (-1, 1):
            w = np.zeros((M, K), np.int8)
            w[m, k] = val
            p = oracle.pack_i2s(w)
            byte, shift = _i2s_byte_and_shift(m, k, K)
            expect = np.full(32 * 512 // 4, 0b01010101, np.uint8)
            expect[byte] = (0b01010101 & ~(3 << shift)) | ((val + 1) << shift)
            assert np.array_equal(p, expect), (m, k)
    # spot values of the formula itself: k = 0, 4, 8, 32 of row 0 and k = 0 of row 1
    assert _i2s_byte_and_shift(0, 0, 256) == (0, 0) and _i2s_byte_and_shift(0, 4, 256) == (4, 0)
    assert _i2s_byte_and_shift(0, 8, 256) == (0, 2) and _i2s_byte_and_shift(0, 32, 256) == (8, 0)
    assert _i2s_byte_and_shift(1, 0, 256) == (64, 0) and _i2s_byte_and_shift(8, 0, 256) == (512, 0)
    assert _i2s_byte_and_shift(16, 0, 256) == (1024, 0) and _i2s_byte_and_shift(0, 256, 512) == (1024, 0)


def test_i2s_blob_read_back_by_the_inverse_statement():
    """The layout stated the other way round: in the 1024-byte piece of 16-row block rb and 256-column chunk c,
    row r of the block owns bytes [64r, 64r+64); there, 32-bit word j (0..15), byte b, bit pair s (bits 8b+2s,
    8b+2s+1 of the word) holds code w+1 of column 256c + 32*(j//2) + 8*s + 4*(j%2) + b.  Every field of a random
    blob (ragged M and K, so padding fields too) is decoded that way."""
    M, K = 21, 448
    w = rand_ternary(M, K)
    p = oracle.pack_i2s(w)
    kp, mp = 512, 32
    assert p.size == mp * kp // 4
    for rb in range(mp // 16):
        for c in range(kp // 256):
            piece = p[rb * 4 * kp + c * 1024: rb * 4 * kp + (c + 1) * 1024]
            for r in range(16):
                for j in range(16):
                    word = int.from_bytes(bytes(piece[64 * r + 4 * j: 64 * r + 4 * j + 4]), "little")
                    for b in range(4):
                        for s_ in range(4):
                            code = (word >> (8 * b + 2 * s_)) & 3
                            m, k = 16 * rb + r, 256 * c + 32 * (j // 2) + 8 * s_ + 4 * (j % 2) + b
                            want = int(w[m, k]) + 1 if (m < M and k < K) else 1
                            assert code == want, (m, k)


def test_i2s_one_hot_dot_products():
    # a single +-1 at position k against q[k] = k - 60 returns exactly +-(k - 60)
    K = 128
    q = (np.arange(K) - 60).astype(np.int8).reshape(1, K)
    w = np.zeros((2 * K, K), np.int8)
    for k in range(K):
        w[2 * k, k] = 1
        w[2 * k + 1, k] = -1
    acc = oracle.i2s_mpgemm(oracle.pack_i2s(w), 2 * K, K, q)
    for k in range(K):
        assert acc[0, 2 * k] == k - 60 and acc[0, 2 * k + 1] == -(k - 60)


def test_i2s_rejects_non_ternary():
    w = np.zeros((1, 128), np.int8)
    w[0, 5] = 2
    with pytest.raises(ValueError):
        oracle.pack_i2s(w)


# ----------------------------------------------------------------------------- TL codes (Tables 4, 5)
def _read_rows(name):
    rows = []
    with open(os.path.join(GOLD, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            rows.append(line.split())
    return rows


def test_tl1_codes_match_table4():
    rows = _read_rows("tl1_table4.txt")
    assert len(rows) == 9
    for w0, w1, code in rows:
        assert oracle.tl1_code(int(w0), int(w1)) == int(code, 2)


def test_tl2_codes_match_table5_and_cover_all_triples():
    rows = _read_rows("tl2_table5.txt")
    assert len(rows) == 9
    for w0, w1, w2, sign, idx in rows:
        c = oracle.tl2_code(int(w0), int(w1), int(w2))
        assert c >> 4 == int(sign) and c & 15 == int(idx, 2)
    seen = {}
    for t in itertools.product((-1, 0, 1), repeat=3):
        c = oracle.tl2_code(*t)
        assert (c & 15) <= 13                              # ceil(27/2) = 14 table entries
        assert c not in seen
        seen[c] = t
        # mirror consolidation: the negated triple has the same index and the opposite sign
        cn = oracle.tl2_code(*[-v for v in t])
        assert (cn & 15) == (c & 15)
        if any(t):
            assert (cn >> 4) != (c >> 4)
    assert oracle.tl2_code(0, 0, 0) == 0
    assert len(seen) == 27


def test_tl_block_fitting_split():
    # ThreeK = floor(K / BK3) * BK3, TwoK = K - ThreeK with BK3 = 96
    for K, three, two in [(3200, 3168, 32), (4096, 4032, 64), (8192, 8160, 32), (14336, 14304, 32),
                          (28672, 28608, 64), (1536, 1536, 0), (8640, 8640, 0)]:
        assert oracle.tl_split("tl2", K) == (three, two)
    assert oracle.tl_split("tl2", 8192, 192) == (8064, 128)
    assert oracle.tl_split("tl1", 8192) == (0, 8192)


def test_tl_sizes_and_bpw():
    # TL2: 5 bits per 3 weights, TL1: 4 bits per 2 weights
    assert oracle.tl_packed_bytes("tl2", 1536, 1536) * 8 * 3 == 5 * 1536 * 1536
    assert oracle.tl_packed_bytes("tl1", 1536, 1536) * 8 == 2 * 1536 * 1536
    assert oracle.tl_packed_bytes("tl2", 32, 8192) == 85 * 640 + 512
    assert oracle.tl_packed_bytes("tl2", 33, 96) == 0 and oracle.tl_packed_bytes("tl2", 32, 97) == 0


@pytest.mark.parametrize("fmt,K", [("tl1", 64), ("tl1", 130), ("tl2", 96), ("tl2", 96 * 2 + 32),
                                   ("tl2", 96 + 64), ("tl2", 34), ("tl2", 96 * 3 + 70)])
def test_tl_round_trip(fmt, K):
    w = rand_ternary(64, K)
    p = oracle.pack_tl(fmt, w)
    assert p.size == oracle.tl_packed_bytes(fmt, 64, K)
    assert np.array_equal(oracle.unpack_tl(fmt, p, 64, K), w)


def test_tl2_documented_byte_positions():
    # one TL2 tile (32 rows x 96 weights).  Row r = g + 8u; triple grp sits in index byte i = grp//2 (grp odd: high
    # nibble) at 64g + 16(i//4) + 4u + i%4; its sign is bit 8(i%4) + 2(i//4) + grp%2 of the word at 512 + 16g + 4u
    w = np.zeros((32, 96), np.int8)
    w[5, 3 * 7: 3 * 7 + 3] = (-1, 1, 0)     # v = -9 + 3 = -6 -> index 6, sign 1; row 5 = (g 5, u 0), byte i = 3
    w[31, 3 * 30: 3 * 30 + 3] = (0, 1, -1)  # v = 2 -> index 2, sign 0; row 31 = (g 7, u 3), byte i = 15
    p = oracle.pack_tl("tl2", w)
    expect = np.zeros(640, np.uint8)
    expect[64 * 5 + 3] = 6 << 4
    expect[512 + 16 * 5 + 3] = 1 << 1       # bit 8*3 + 2*0 + 1 = 25
    expect[64 * 7 + 16 * 3 + 4 * 3 + 3] = 2
    assert np.array_equal(p, expect)


def test_tl2_tile_read_back_by_the_inverse_statement():
    """The layout stated the other way round -- which (row, triple) a byte / a sign bit of the tile holds: byte p of
    the index plane holds index byte 4*((p%64)//16) + p%4 of row p//64 + 8*((p%16)//4); bit b of the sign word at
    512 + 4*s holds the sign of triple 2*(4*((b%8)//2) + b//8) + b%2 of row s//4 + 8*(s%4).  Every position of a
    random tile is decoded that way and compared with the codes of Table 5 computed from the weights."""
    w = rand_ternary(32, 96)
    p = oracle.pack_tl("tl2", w)
    v = 9 * w[:, 0::3].astype(int) + 3 * w[:, 1::3] + w[:, 2::3]          # [32][32]
    for pos in range(512):
        row, i = pos // 64 + 8 * ((pos % 16) // 4), 4 * ((pos % 64) // 16) + pos % 4
        assert p[pos] & 15 == abs(v[row, 2 * i]) and p[pos] >> 4 == abs(v[row, 2 * i + 1])
    for s_ in range(32):
        word = int.from_bytes(bytes(p[512 + 4 * s_: 516 + 4 * s_]), "little")
        row = s_ // 4 + 8 * (s_ % 4)
        for b in range(32):
            grp = 2 * (4 * ((b % 8) // 2) + b // 8) + b % 2
            assert (word >> b) & 1 == int(v[row, grp] < 0)


def test_tl1_documented_byte_positions_and_padding():
    w = np.zeros((32, 34), np.int8)         # 17 pairs, tile padded to 32 pairs with code 4
    w[2, 0:2] = (1, -1)                     # code 6, pair 0 -> low nibble of index byte 0 of row 2 = (g 2, u 0)
    w[2, 32:34] = (-1, -1)                  # code 0, pair 16 -> low nibble of index byte 8 (word 2, byte 0)
    w[26, 2:4] = (1, 1)                     # code 8, pair 1 -> high nibble of index byte 0 of row 26 = (g 2, u 3)
    p = oracle.pack_tl("tl1", w)
    expect = np.full(512, 0x44, np.uint8)
    expect[64 * 2 + 0] = 0x46
    expect[64 * 2 + 16 * 2 + 0] = 0x40
    expect[64 * 2 + 4 * 3 + 0] = 0x84
    assert np.array_equal(p, expect)


def test_dequant_segments_closed_form():
    """Two stacked matrices with scales 0.5 and 3: powers of two and small integers keep every product exact, so the
    expected values are written down; a single segment equals oracle.dequant; bad segment lists are refused."""
    acc = np.array([[2, -4, 6, 8, -10], [1, 1, 1, 1, 1]], np.int32)
    act_scale = np.array([0.25, 2.0], np.float32)
    y = oracle.dequant_segments(acc, act_scale, [2, 5], [0.5, 3.0])
    assert np.array_equal(y, np.array([[0.25, -0.5, 4.5, 6.0, -7.5], [1.0, 1.0, 6.0, 6.0, 6.0]]))
    assert np.array_equal(oracle.dequant_segments(acc, act_scale, [5], [0.75]), oracle.dequant(acc, act_scale, 0.75))
    for bad in ([2, 4], [3, 3, 5], [6]):
        with pytest.raises(Exception):
            oracle.dequant_segments(acc, act_scale, bad, [1.0] * len(bad))


# ----------------------------------------------------------------------------- LUT build (Alg. 3 / Alg. 4 PreCompute)
def test_lut_identities():
    q = rand_q(1, 96 * 2 + 64)[0]
    lut = oracle.tl_build_lut("tl2", q)
    assert lut.shape == (64 + 32, 16)
    for g in range(64):
        a0, a1, a2 = (int(v) for v in q[3 * g: 3 * g + 3])
        e = lut[g]
        assert e[0] == 0 and e[1] == a2 and e[3] == a1 and e[9] == a0 and e[13] == a0 + a1 + a2
        assert e[2] == a1 - a2 and e[4] == a1 + a2 and e[14] == 0 and e[15] == 0
        assert np.abs(e).max() <= 384
        for i in range(14):                  # every entry = dot with the balanced-ternary digits of i
            d0 = round(i / 9)
            d1 = round((i - 9 * d0) / 3)
            d2 = i - 9 * d0 - 3 * d1
            assert {d0, d1, d2} <= {-1, 0, 1}
            assert e[i] == d0 * a0 + d1 * a1 + d2 * a2
    for p in range(32):
        a0, a1 = int(q[192 + 2 * p]), int(q[192 + 2 * p + 1])
        e = lut[64 + p]
        assert e[4] == 0 and all(e[i] + e[8 - i] == 0 for i in range(9))
        assert e[8] == a0 + a1 and e[6] == a0 - a1 and e[5] == a1 and e[7] == a0
        assert not e[9:].any()


# ----------------------------------------------------------------------------- whole mpGEMM: invariants, cross-format equality
@pytest.mark.parametrize("K", [128, 96 * 2 + 32, 96 * 4 + 64, 576])
def test_all_formats_give_the_definition(K):
    T, M = 3, 64
    q, w = rand_q(T, K), rand_ternary(M, K, 0.4)
    ref = q.astype(np.int64) @ w.astype(np.int64).T
    assert np.array_equal(oracle.mpgemm_def(q, w), ref)
    if K % 64 == 0:
        assert np.array_equal(oracle.i2s_mpgemm(oracle.pack_i2s(w), M, K, q), ref)
    assert np.array_equal(oracle.tl_mpgemm("tl1", oracle.pack_tl("tl1", w), M, K, q), ref)
    assert np.array_equal(oracle.tl_mpgemm("tl2", oracle.pack_tl("tl2", w), M, K, q), ref)


def test_constant_weight_invariants():
    T, M, K = 2, 32, 96 * 3 + 32
    q = rand_q(T, K)
    sums = q.astype(np.int64).sum(axis=1)
    for val in (0, 1, -1):
        w = np.full((M, K), val, np.int8)
        for acc in (oracle.mpgemm_def(q, w),
                    oracle.tl_mpgemm("tl2", oracle.pack_tl("tl2", w), M, K, q),
                    oracle.tl_mpgemm("tl1", oracle.pack_tl("tl1", w), M, K, q)):
            assert np.array_equal(acc, np.repeat((val * sums)[:, None], M, axis=1))


def test_tl2_one_hot_across_split_and_tile_boundaries():
    K = 96 * 2 + 64                      # two TL2 tiles then one TL1 tile
    q = ((np.arange(K) % 251) - 125).astype(np.int8).reshape(1, K)
    probes = [0, 1, 2, 94, 95, 96, 97, 191, 192, 193, 254, 255]
    w = np.zeros((32, K), np.int8)
    for i, k in enumerate(probes):
        w[i, k] = 1 if i % 2 == 0 else -1
    acc = oracle.tl_mpgemm("tl2", oracle.pack_tl("tl2", w), 32, K, q)
    for i, k in enumerate(probes):
        assert acc[0, i] == (1 if i % 2 == 0 else -1) * int(q[0, k])
    assert not acc[0, len(probes):].any()


# ----------------------------------------------------------------------------- ELUT beyond ternary (App. A)
def rand_alphabet(M, K, C):
    return rng.integers(-(C // 2), -(C // 2) + C, size=(M, K)).astype(np.int8)


def test_elut_bits_per_weight_match_table3():
    rows = _read_rows("elut_table3.txt")
    assert len(rows) == 3
    for C, g, bpw_b, bpw_e in rows:
        C, g = int(C), int(g)
        assert oracle.elut_bitwise_bits(C) == int(bpw_b)
        assert round(oracle.elut_index_bits(C, g) / g, 2) == float(bpw_e)
    # a group index needs the smallest b with 2^b >= C^g
    for C, g in itertools.product(range(2, 9), range(1, 5)):
        b = oracle.elut_index_bits(C, g)
        assert 2 ** b >= C ** g > 2 ** (b - 1) or (C ** g == 1 and b == 0)


def test_elut_alphabet_and_index_are_base_c_digits():
    assert [oracle.elut_lo(C) for C in (2, 3, 4, 5, 8)] == [-1, -1, -2, -2, -4]
    for C, g in [(3, 2), (3, 3), (4, 2), (5, 2), (4, 3), (3, 5)]:
        lo = -(C // 2)
        seen = set()
        for grp in itertools.product(range(lo, lo + C), repeat=g):
            want = 0
            for wv in grp:                       # Horner, first weight most significant
                want = want * C + (wv - lo)
            got = oracle.elut_index(grp, C)
            assert got == want
            seen.add(got)
        assert seen == set(range(C ** g))        # a bijection onto [0, C^g)
        assert oracle.elut_index([lo - 1] + [0] * (g - 1), C) == -1
        assert oracle.elut_index([0] * (g - 1) + [lo + C], C) == -1
    # the all-zero group sits in the middle of the odd alphabets' range
    assert oracle.elut_index([0, 0], 5) == 12 and oracle.elut_index([0, 0], 4) == 10 and oracle.elut_index([0, 0], 3) == 4


def test_elut_ternary_pairs_are_table4_and_triples_are_table5():
    for w0, w1, code in _read_rows("tl1_table4.txt"):
        assert oracle.elut_index([int(w0), int(w1)], 3) == int(code, 2)
    # Table 5 is the mirror-consolidated form of the 27-entry table: v = index - 13, |v| its index, v < 0 its sign
    for w0, w1, w2, sign, idx in _read_rows("tl2_table5.txt"):
        v = oracle.elut_index([int(w0), int(w1), int(w2)], 3) - 13
        assert abs(v) == int(idx, 2) and int(v < 0) == int(sign)


@pytest.mark.parametrize("C,g", [(3, 2), (3, 3), (4, 2), (5, 2), (4, 3), (5, 3), (3, 5), (16, 2)])
def test_elut_table_setup_entries_by_brute_force(C, g):
    K = 6 * g
    q = rand_q(1, K)[0]
    lut = oracle.elut_table_setup(q, C, g)
    assert lut.shape == (K // g, C ** g)
    lo = -(C // 2)
    for k in range(K // g):
        a = [int(v) for v in q[g * k: g * k + g]]
        for i, grp in enumerate(itertools.product(range(lo, lo + C), repeat=g)):   # lexicographic = index order
            assert lut[k, i] == sum(wv * av for wv, av in zip(grp, a))
        zero = oracle.elut_index([0] * g, C)
        assert lut[k, zero] == 0
        if C % 2 == 1:                           # symmetric alphabet: the table is odd about its middle
            assert all(lut[k, i] + lut[k, C ** g - 1 - i] == 0 for i in range(C ** g))


def test_elut_tables_reduce_to_the_ternary_ones():
    q = rand_q(1, 96 * 2)[0]
    pair = oracle.elut_table_setup(q, 3, 2)
    tl1 = oracle.tl_build_lut("tl1", q)                   # Alg. 3 PreCompute, 9 of 16 slots used
    assert np.array_equal(pair, tl1[: pair.shape[0], :9])
    triple = oracle.elut_table_setup(q, 3, 3)
    tl2 = oracle.tl_build_lut("tl2", q)                   # Alg. 4 PreCompute: the non-negative half
    for v in range(-13, 14):
        assert np.array_equal(triple[:, 13 + v], np.sign(v) * tl2[:, abs(v)] if v else tl2[:, 0])


@pytest.mark.parametrize("C,g,K", [(3, 2, 64), (3, 3, 96), (4, 2, 130), (5, 2, 70), (5, 3, 99), (4, 4, 64), (3, 5, 80)])
def test_elut_lookup_accumulation_gives_the_definition(C, g, K):
    T, M = 3, 40
    q, w = rand_q(T, K), rand_alphabet(M, K, C)
    ref = q.astype(np.int64) @ w.astype(np.int64).T
    assert np.array_equal(oracle.mpgemm_def(q, w), ref)
    idx = oracle.elut_encode(w, C, g)
    assert idx.max() < C ** g
    assert np.array_equal(oracle.elut_mpgemm(idx, K, C, g, q), ref)
    bad = w.copy()
    bad[0, 0] = -(C // 2) + C
    with pytest.raises(ValueError):
        oracle.elut_encode(bad, C, g)


@pytest.mark.parametrize("C", [3, 4, 5])
def test_elut2_blob_size_round_trip_and_definition(C):
    # 4 bits per pair for C <= 4, 5 bits for C = 5: 2 and 2.5 bits per weight (Table 3)
    assert oracle.elut2_packed_bytes(C, 64, 128) * 8 == (5 if C == 5 else 4) * 64 * 128 // 2
    assert oracle.elut2_packed_bytes(C, 33, 64) == 0 and oracle.elut2_packed_bytes(C, 32, 65) == 0
    assert oracle.elut2_packed_bytes(6, 32, 64) == 0
    for K in (64, 130, 2, 192 + 34):
        T, M = 2, 64
        q, w = rand_q(T, K), rand_alphabet(M, K, C)
        p = oracle.pack_elut2(C, w)
        assert p.size == oracle.elut2_packed_bytes(C, M, K) == (M // 32) * ((K + 63) // 64) * (640 if C == 5 else 512)
        assert np.array_equal(oracle.unpack_elut2(C, p, M, K), w)
        assert np.array_equal(oracle.elut2_mpgemm(C, p, M, K, q), q.astype(np.int64) @ w.astype(np.int64).T)
    with pytest.raises(ValueError):
        oracle.pack_elut2(C, np.full((32, 64), -(C // 2) - 1, np.int8))


def test_elut2_ternary_blob_is_the_tl1_blob():
    w = rand_ternary(64, 192 + 34)
    assert np.array_equal(oracle.pack_elut2(3, w), oracle.pack_tl("tl1", w))


def test_elut2_documented_byte_positions():
    """C = 5: pair grp of row r = g + 8u has index 5(w0+2) + (w1+2); its low four bits sit in the nibble of index
    byte i = grp//2 (grp odd: high nibble) at 64g + 16(i//4) + 4u + i%4, its fifth bit at bit 8(i%4) + 2(i//4) + grp%2
    of the word at 512 + 16g + 4u.  Zero weights have index 12: every other nibble is 0xC, every other high bit 0."""
    w = np.zeros((32, 64), np.int8)
    w[5, 14:16] = (2, 1)        # index 23 = 16 + 7: row 5 = (g 5, u 0), pair 7 -> byte i = 3, high nibble; bit 8*3+0+1
    w[31, 60:62] = (-2, -1)     # index 1: row 31 = (g 7, u 3), pair 30 -> byte i = 15, low nibble
    w[9, 0:2] = (1, 2)          # index 19 = 16 + 3: row 9 = (g 1, u 1), pair 0 -> byte 0, low nibble; bit 0
    p = oracle.pack_elut2(5, w)
    expect = np.zeros(640, np.uint8)
    expect[:512] = 0xCC
    expect[64 * 5 + 3] = 0x7C
    expect[512 + 16 * 5 + 3] = 1 << 1
    expect[64 * 7 + 16 * 3 + 4 * 3 + 3] = 0xC1
    expect[64 * 1 + 4 * 1] = 0xC3
    expect[512 + 16 * 1 + 4 * 1] = 1
    assert np.array_equal(p, expect)
    # C = 4: index 4(w0+2) + (w1+2), four bits, no second plane; zero weights have index 10
    w4 = np.zeros((32, 34), np.int8)
    w4[2, 0:2] = (1, -2)        # index 12
    w4[26, 2:4] = (-2, 1)       # index 3: row 26 = (g 2, u 3), pair 1 -> high nibble of byte 0
    p4 = oracle.pack_elut2(4, w4)
    expect4 = np.full(512, 0xAA, np.uint8)
    expect4[64 * 2] = 0xAC
    expect4[64 * 2 + 4 * 3] = 0x3A
    assert np.array_equal(p4, expect4)


@pytest.mark.parametrize("C", [4, 5])
def test_elut2_one_hot_dot_products(C):
    # a single non-zero weight v at column k against q[k] returns exactly v * q[k], for every column of two tiles
    K = 128
    q = ((np.arange(K) * 7) % 251 - 125).astype(np.int8).reshape(1, K)
    lo = -(C // 2)
    vals = [v for v in range(lo, lo + C) if v != 0]
    rows = [(k, v) for k in range(K) for v in vals]
    M = ((len(rows) + 31) // 32) * 32
    w = np.zeros((M, K), np.int8)
    for i, (k, v) in enumerate(rows):
        w[i, k] = v
    acc = oracle.elut2_mpgemm(C, oracle.pack_elut2(C, w), M, K, q)
    for i, (k, v) in enumerate(rows):
        assert acc[0, i] == v * int(q[0, k])
    assert not acc[0, len(rows):].any()

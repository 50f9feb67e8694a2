"""bitnet_linear_group (a list of linears in one persistent kernel) against the CPU oracle, through the
C ABI: quantised codes, scale bit patterns and int32 accumulators identical, fp32 outputs within 1e-6."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth

from helpers import Guarded, check_y, npy

pytestmark = pytest.mark.gpu


def tern(seed, M, K, p0=1 / 3, pp=1 / 3):
    return synth.ternary(seed, 77, M, K, p0, pp)


class Item:
    """One linear of a group: weights, activations and guarded output buffers."""

    def __init__(self, fmt, M, K, T, seed, x=None, w_scale=0.75):
        self.fmt, self.M, self.K, self.T, self.w_scale = fmt, M, K, T, w_scale
        self.w = tern(seed, M, K)
        self.x = synth.normal(seed, 1000 + T, T, K) if x is None else x
        self.xd = self.x.cuda()
        self.blob = bn.pack(fmt, self.w.cuda())
        self.gq, self.gsc = Guarded((T, K), torch.int8), Guarded((T,), torch.float32)
        self.gy, self.gacc = Guarded((T, M), torch.float32), Guarded((T, M), torch.int32)
        self.ws = bn.new_workspace(fmt, T, M, K)

    def desc(self):
        return dict(fmt=self.fmt, packed=self.blob, w_scale=self.w_scale, M=self.M, K=self.K, x=self.xd, q=self.gq.t,
                    act_scale=self.gsc.t, y=self.gy.t, acc_out=self.gacc.t, workspace=self.ws)

    def check(self, rows=None):
        for name, g in (("q", self.gq), ("act_scale", self.gsc), ("y", self.gy), ("acc", self.gacc)):
            assert g.intact(), f"M={self.M} K={self.K} T={self.T}: bytes outside {name} were written"
        q_ref, sc_ref, _ = oracle.quant_act(self.x.numpy())
        assert np.array_equal(npy(self.gq.t), q_ref)
        assert np.array_equal(npy(self.gsc.t).view(np.uint32), sc_ref.view(np.uint32))
        w = self.w.numpy()
        acc, y = npy(self.gacc.t), self.gy.t
        if rows is not None:
            w, acc, y = w[rows], acc[:, rows], y[:, rows]
        acc_ref = oracle.mpgemm_def(q_ref, np.ascontiguousarray(w))
        assert np.array_equal(acc, acc_ref)
        check_y(y, acc_ref, sc_ref, self.w_scale)


def run_group(items):
    grp = bn.make_group([it.desc() for it in items])
    bn.bitnet_linear_group(grp)
    torch.cuda.synchronize()
    assert bn.bitnet_device_status() == 0


def test_group_small_ragged_list():
    """Few units for the SMs, ragged row counts, K with a padded last chunk, every token count, one item per
    shape class; most CTAs get no work or a single unit, and units of neighbouring items share a CTA."""
    shapes = [(1, 1024, 1), (7, 1536, 2), (300, 3200, 3), (33, 8640, 4), (160, 2048, 5), (48, 28672, 1),
              (100, 8192, 8), (16, 1024, 6), (17, 4096, 7)]
    items = [Item("i2s", M, K, T, 100 + i) for i, (M, K, T) in enumerate(shapes)]
    run_group(items)
    for it in items:
        it.check()


WIDE_SHAPES = [(40, 2048, 9), (300, 8192, 16), (33, 28672, 12), (64, 4096, 3), (1000, 3200, 13), (64, 4096, 17),
               (17, 1536, 10), (2000, 1024, 11), (160, 28672, 16), (48, 16384, 14), (16, 8192, 15), (640, 4096, 8)]


def test_group_nine_to_sixteen_tokens():
    """Items with 9 to 16 tokens run through the grouped kernel's two-group form (launches of their own, between those
    of the neighbours with up to 8 tokens): every token count, ragged rows, long rows walked in parts, an item with 17
    tokens (left to the streaming or mid-batch kernel) in between."""
    items = [Item("i2s", M, K, T, 150 + i) for i, (M, K, T) in enumerate(WIDE_SHAPES)]
    run_group(items)
    for it in items:
        it.check()


def test_group_nine_to_sixteen_tokens_shared_input_and_many_units():
    """Two-group form: linears that share their input (quantised once per CTA, codes stored per item), and enough units
    that every warp takes whole units and walks several of them."""
    x = synth.normal(170, 3, 12, 4096)
    items = [Item("i2s", 4096, 4096, 12, 171, x=x), Item("i2s", 1024, 4096, 12, 172, x=x), Item("i2s", 11008, 4096, 12, 173, x=x),
             Item("i2s", 40000, 2048, 16, 174)]
    items[1].xd = items[2].xd = items[0].xd
    run_group(items)
    for it in items:
        it.check(rows=np.unique(np.concatenate([[0, 15, 16, it.M - 1], np.random.default_rng(it.M).integers(0, it.M, 200)])))


@pytest.mark.parametrize("extra", [dict(BITNET_GROUP_WIDE="0"), dict(BITNET_GROUP_S="1"),
                                   dict(BITNET_GROUP_S="2", BITNET_GROUP_DEPTH="8")])
def test_group_nine_to_sixteen_tokens_switches_in_child_processes(extra):
    """Read-once switches on the list of 9-to-16-token items: BITNET_GROUP_WIDE=0 runs such items as two items of the
    one-group kernel over the same weights (tokens 0..7, then the rest); BITNET_GROUP_S=1 forces one warp per unit
    (the form with one buffer of partial sums per warp and the fewest parts of K, which otherwise only launches with
    thousands of units take); two warps per unit with rings of eight chunks."""
    import os
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, 'tests')\n"
        "import paper_2502_11880_b200 as bn\n"
        "from test_gpu_group import Item, run_group, WIDE_SHAPES\n"
        "items = [Item('i2s', M, K, T, 150 + i) for i, (M, K, T) in enumerate(WIDE_SHAPES)]\n"
        "run_group(items)\n"
        "for it in items: it.check()\n"
        "assert bn.bitnet_device_status() == 0\n"
        "print('ok')\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, **extra), capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0 and "ok" in out.stdout, (extra, out.stderr[-2000:])


def test_group_nine_to_sixteen_tokens_one_warp_per_unit():
    """Enough units that the launch runs with one warp per unit by itself: the two-group form with one buffer of
    partial sums per warp, K = 8192 in one part at 16 tokens."""
    items = [Item("i2s", 160000, 1024, 12, 176), Item("i2s", 4096, 8192, 16, 177), Item("i2s", 1024, 28672, 16, 178)]
    run_group(items)
    for it in items:
        it.check(rows=np.unique(np.concatenate([[0, 15, 16, it.M - 1], np.random.default_rng(it.M).integers(0, it.M, 150)])))


def test_group_many_units_per_cta_and_shared_inputs():
    """More units than warp groups (every group walks several units and crosses item borders), Q/K/V-like items
    that share one activation buffer (quantised once, each item still gets its codes), and an item whose token
    count differs from its neighbours'."""
    K = 4096
    x = synth.normal(7, 1, 2, K)
    items = [Item("i2s", 6144, K, 2, 200, x=x), Item("i2s", 4096, K, 2, 201, x=x), Item("i2s", 5000, K, 2, 202, x=x),
             Item("i2s", 4096, 14336, 1, 203), Item("i2s", 9000, 2048, 3, 204)]
    # the first two share the device input AND the code buffers, the third only the input
    items[1].xd = items[0].xd
    items[2].xd = items[0].xd
    d = [it.desc() for it in items]
    d[1]["q"], d[1]["act_scale"] = d[0]["q"], d[0]["act_scale"]
    grp = bn.make_group(d)
    bn.bitnet_linear_group(grp)
    torch.cuda.synchronize()
    items[1].gq, items[1].gsc = items[0].gq, items[0].gsc
    for it in items:
        it.check()


def test_group_mixed_formats_fall_back_in_order():
    """TL2 items, a prefill-sized item and a short-K item inside the list are run by bitnet_linear; the I2_S decode
    items on either side still go through the grouped kernel."""
    items = [Item("i2s", 64, 2048, 1, 300), Item("tl2", 64, 3200, 2, 301), Item("i2s", 96, 8192, 2, 302),
             Item("i2s", 32, 256, 1, 303), Item("i2s", 64, 1536, 24, 304), Item("tl1", 32, 130, 1, 305),
             Item("i2s", 200, 4096, 4, 306)]
    run_group(items)
    for it in items:
        it.check()


def test_group_more_items_than_the_small_argument_block():
    """60 items: the kernel instance with the 32 KB argument block."""
    items = [Item("i2s", 16 * (1 + i % 5), 1024 + 256 * (i % 3), 1 + i % 2, 400 + i) for i in range(60)]
    run_group(items)
    for it in items:
        it.check()


@pytest.mark.parametrize("fmt,count", [("i2s", 430), ("tl2", 360), ("tl1", 350)])
def test_group_more_items_than_one_launch_takes(fmt, count):
    """More items than the largest argument block holds (409 for I2_S, 340 for the scan kernel): the call is cut into
    several launches, in list order."""
    items = [Item(fmt, 32 * (1 + i % 3), 1024 + 256 * (i % 3), 1 + i % 3, 3000 + i) for i in range(count)]
    run_group(items)
    for it in items:
        it.check()


def test_group_equals_single_calls_and_given_workload_layer():
    """A 100B-shaped decoder layer (8192->10240, 8192->8192, 8192->57344, 28672->8192) at one token through the
    grouped call: every output row against the oracle."""
    wl = synth.CONFIGS["sweep100b"]
    items = []
    for j, lin in enumerate(wl.linears):
        it = Item.__new__(Item)
        it.fmt, it.M, it.K, it.T = "i2s", lin.M, lin.K, 1
        it.w = wl.weights(3, j)
        it.w_scale = synth.absmean_scale(it.w)
        it.x = wl.activations(3, j, 1)
        it.xd = it.x.cuda()
        it.blob = bn.pack("i2s", it.w.cuda())
        it.gq, it.gsc = Guarded((1, lin.K), torch.int8), Guarded((1,), torch.float32)
        it.gy, it.gacc = Guarded((1, lin.M), torch.float32), Guarded((1, lin.M), torch.int32)
        it.ws = None
        items.append(it)
    run_group(items)
    for it in items:
        it.check()
    # and the same list through bitnet_linear, one call per item: identical bits
    for it in items:
        y, q, sc, acc = bn.bitnet_linear("i2s", it.blob, it.w_scale, it.M, it.K, it.xd, want_acc=True)
        torch.cuda.synchronize()
        assert torch.equal(y, it.gy.t) and torch.equal(acc, it.gacc.t) and torch.equal(q, it.gq.t)


@pytest.mark.parametrize("T", [2, 4])
def test_group_layer_batched(T):
    """The 8B-shaped layer at 2 and 4 tokens per linear through the grouped call, sampled rows."""
    wl = synth.CONFIGS["layer8b"]
    items = [Item("i2s", lin.M, lin.K, T, 500 + j) for j, lin in enumerate(wl.linears)]
    run_group(items)
    rng = np.random.default_rng(5)
    for it in items:
        it.check(rows=np.sort(rng.choice(it.M, 200, replace=False)))


def test_group_rejects_malformed_items():
    it = Item("i2s", 32, 1024, 1, 600)
    d = it.desc()
    grp = bn.make_group([d])
    grp[0].K = 1000                      # not a multiple of 64
    with pytest.raises(bn.BitnetError, match="shape"):
        bn.bitnet_linear_group(grp)
    grp = bn.make_group([d])
    grp[0].y = None
    with pytest.raises(bn.BitnetError, match="invalid"):
        bn.bitnet_linear_group(grp)


def test_group_tl2_items_through_the_scan_kernel():
    """TL2 items (decode table + tensor cores): block-fitting splits with no, one and two pair tiles in the tail,
    every token count, rows a multiple of 32 only, items sharing an input, an I2_S item in between."""
    x = synth.normal(9, 1, 2, 4096)
    items = [Item("tl2", 64, 96 * 12, 1, 700), Item("tl2", 320, 3200, 3, 701), Item("tl2", 96, 8640, 4, 702),
             Item("tl2", 4096, 4096, 2, 703, x=x), Item("tl2", 2048, 4096, 2, 704, x=x), Item("i2s", 64, 2048, 1, 705),
             Item("tl2", 32, 8192, 8, 706), Item("tl2", 160, 28672, 1, 707), Item("tl2", 64, 96 * 20 + 92, 5, 708)]
    items[4].xd = items[3].xd
    run_group(items)
    for it in items:
        it.check()


def test_group_tl1_items_through_the_scan_kernel():
    """TL1 items: a TL1 blob is the pair-index blob of cardinality 3, so decode batches run in the scan kernel's pair
    mode (the index byte of two pairs selects a table entry holding their four weights).  Ragged last tiles, every
    token count, items sharing an input, a TL2 and an I2_S item in between, a row too short for the kernel."""
    x = synth.normal(9, 2, 2, 4096)
    items = [Item("tl1", 64, 64 * 12, 1, 720), Item("tl1", 320, 3200, 3, 721), Item("tl1", 96, 8640, 4, 722),
             Item("tl1", 4096, 4096, 2, 723, x=x), Item("tl1", 2048, 4096, 2, 724, x=x), Item("tl2", 64, 2048, 1, 725),
             Item("tl1", 32, 8192, 8, 726), Item("tl1", 160, 28672, 1, 727), Item("i2s", 64, 2048, 1, 728),
             Item("tl1", 64, 64 * 20 + 36, 5, 729), Item("tl1", 64, 128, 2, 730), Item("tl1", 32, 28672, 8, 731)]
    items[4].xd = items[3].xd
    run_group(items)
    for it in items:
        it.check()


def test_group_tl2_workload_layer():
    """A 100B-shaped decoder layer in the TL2 encoding at one token through the grouped call (one persistent scan
    kernel): sampled rows of every linear against the oracle, and the whole vectors against the I2_S result."""
    wl = synth.CONFIGS["sweep100b"]
    rng = np.random.default_rng(11)
    for j, lin in enumerate(wl.linears):
        wd = wl.weights(5, j, device="cuda")
        x = wl.activations(5, j, 1)
        rows = np.unique(np.concatenate([[0, 31, 32, lin.M - 1], rng.integers(0, lin.M, 96)]))
        w_rows = np.stack([wl.weights(5, j, row_start=int(r), rows=1).numpy()[0] for r in rows])
        outs = {}
        for fmt in ("tl2", "i2s"):
            blob = bn.pack(fmt, wd, check=False)
            q = torch.empty((1, lin.K), dtype=torch.int8, device="cuda")
            sc = torch.empty(1, dtype=torch.float32, device="cuda")
            y = torch.empty((1, lin.M), dtype=torch.float32, device="cuda")
            acc = torch.empty((1, lin.M), dtype=torch.int32, device="cuda")
            grp = bn.make_group([dict(fmt=fmt, packed=blob, w_scale=0.625, M=lin.M, K=lin.K, x=x.cuda(), q=q, act_scale=sc,
                                      y=y, acc_out=acc)])
            bn.bitnet_linear_group(grp)
            torch.cuda.synchronize()
            outs[fmt] = (y, acc, q, sc)
            del blob
        y, acc, q, sc = outs["tl2"]
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(q), q_ref)
        acc_ref = oracle.mpgemm_def(q_ref, np.ascontiguousarray(w_rows))
        assert np.array_equal(npy(acc)[:, rows], acc_ref)
        check_y(y[:, torch.as_tensor(rows).cuda()], acc_ref, sc_ref, 0.625)
        assert torch.equal(acc, outs["i2s"][1]) and torch.equal(y, outs["i2s"][0])
        del wd
        torch.cuda.empty_cache()
    assert bn.bitnet_device_status() == 0


def test_group_long_rows_walked_in_parts():
    """Batches whose staged codes of a whole row do not fit in shared memory: the CTA walks the item's K in two or
    three parts, the integer sums resting in y between the parts.  Part sizes that do not divide the row evenly, a
    ragged last 16-row unit, several units per warp group, and neighbours of other shapes on either side."""
    shapes = [(40, 2048, 2), (1000, 28672, 8), (70, 29440, 8), (520, 28672, 5), (33, 14336, 8), (48, 28672, 6), (64, 8192, 8)]
    items = [Item("i2s", M, K, T, 800 + i) for i, (M, K, T) in enumerate(shapes)]
    run_group(items)
    for it in items:
        it.check()
    # the same list once more into the same buffers (y held integer scratch in between: no stale state may survive)
    run_group(items)
    for it in items:
        it.check()


def test_workload_sweep100b_every_layer_sampled_rows():
    """All 80 layers of the 100B-shaped sweep, both encodings: weights drawn and packed in device memory as the
    benchmark does, each layer's eight linears (four per format) in one grouped call; about a hundred output rows
    per tensor are recomputed by the oracle from host re-draws of the same weights, and the TL2 accumulators must
    equal the I2_S ones everywhere."""
    wl = synth.CONFIGS["sweep100b"]
    nl = len(wl.linears)
    bufs = {}
    for fmt in ("i2s", "tl2"):
        for j, lin in enumerate(wl.linears):
            bufs[fmt, j] = (torch.empty((1, lin.K), dtype=torch.int8, device="cuda"), torch.empty(1, dtype=torch.float32, device="cuda"),
                            torch.empty((1, lin.M), dtype=torch.float32, device="cuda"),
                            torch.empty((1, lin.M), dtype=torch.int32, device="cuda"))
    for layer in range(wl.layers):
        rng = np.random.default_rng(7000 + layer)
        items, xs, blobs = [], [], []
        for fmt in ("i2s", "tl2"):
            for j, lin in enumerate(wl.linears):
                wd = wl.weights(layer, j, device="cuda")
                blobs.append(bn.pack(fmt, wd, check=False))
                del wd
                if fmt == "i2s":
                    xs.append(wl.activations(layer, j, 1))
                q, sc, y, acc = bufs[fmt, j]
                items.append(dict(fmt=fmt, packed=blobs[-1], w_scale=0.625, M=lin.M, K=lin.K, x=xs[j].cuda(), q=q,
                                  act_scale=sc, y=y, acc_out=acc))
        bn.bitnet_linear_group(bn.make_group(items))
        torch.cuda.synchronize()
        for j, lin in enumerate(wl.linears):
            rows = np.unique(np.concatenate([[0, 15, 16, 31, 32, lin.M - 1], rng.integers(0, lin.M, 96)]))
            w_rows = np.stack([wl.weights(layer, j, row_start=int(r), rows=1).numpy()[0] for r in rows])
            q_ref, sc_ref, _ = oracle.quant_act(xs[j].numpy())
            acc_ref = oracle.mpgemm_def(q_ref, np.ascontiguousarray(w_rows))
            rows_d = torch.as_tensor(rows).cuda()
            for fmt in ("i2s", "tl2"):
                q, sc, y, acc = bufs[fmt, j]
                assert np.array_equal(npy(q), q_ref), (layer, j, fmt)
                assert np.array_equal(npy(sc).view(np.uint32), sc_ref.view(np.uint32))
                assert np.array_equal(npy(acc[:, rows_d]), acc_ref), (layer, j, fmt)
                check_y(y[:, rows_d], acc_ref, sc_ref, 0.625)
            assert torch.equal(bufs["tl2", j][3], bufs["i2s", j][3]), (layer, j)
            assert torch.equal(bufs["tl2", j][2], bufs["i2s", j][2]), (layer, j)
        del items, blobs
    assert bn.bitnet_device_status() == 0


@pytest.mark.parametrize("fmt,T", [("i2s", 1), ("i2s", 3), ("i2s", 12), ("tl2", 1), ("tl2", 2), ("tl1", 1)])
def test_linear_segments_fused_qkv_and_gate_up(fmt, T):
    """The 8B-shaped layer with its fused tensors as the model keeps them: Q/K/V stacked (4096 + 1024 + 1024 rows,
    three scales) and gate/up stacked (2 x 14336 rows, two scales), one call each; every accumulator against the
    definition and every output against the oracle's per-segment rescale.  12 tokens and TL1 take the fallback
    (whole tensor, then a rescale of the segments' columns)."""
    for (M, K, ends, scales, seed) in [(6144, 4096, [4096, 5120, 6144], [0.5, 0.71875, 0.4375], 1000),
                                       (28672, 4096, [14336, 28672], [0.625, 0.6875], 1001),
                                       (200, 2048, [64, 128, 200] if fmt == "i2s" else [64, 128, 192], [1.0, 0.25, 3.0], 1002)]:
        M = ends[-1]
        w = tern(seed, M, K, 0.4, 0.3)
        x = synth.normal(seed, 2000 + T, T, K)
        blob = bn.pack(fmt, w.cuda())
        gq, gsc = Guarded((T, K), torch.int8), Guarded((T,), torch.float32)
        gy, gacc = Guarded((T, M), torch.float32), Guarded((T, M), torch.int32)
        bn.bitnet_linear_segments(fmt, blob, M, K, ends, scales, x.cuda(), q=gq.t, act_scale=gsc.t, y=gy.t, acc_out=gacc.t)
        torch.cuda.synchronize()
        for name, g in (("q", gq), ("act_scale", gsc), ("y", gy), ("acc", gacc)):
            assert g.intact(), name
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(gq.t), q_ref)
        assert np.array_equal(npy(gsc.t).view(np.uint32), sc_ref.view(np.uint32))
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(gacc.t), acc_ref)
        y_ref = oracle.dequant_segments(acc_ref, sc_ref, ends, scales)
        y = npy(gy.t).astype(np.float64)
        assert np.all(np.abs(y - y_ref) <= 1e-6 * np.abs(y_ref))
        assert np.all(y[acc_ref == 0] == 0.0)
    assert bn.bitnet_device_status() == 0


def test_linear_segments_rejects_bad_lists():
    w = tern(1100, 64, 1024)
    blob = bn.pack("i2s", w.cuda())
    x = synth.normal(1100, 1, 1, 1024).cuda()
    with pytest.raises(bn.BitnetError, match="shape"):
        bn.bitnet_linear_segments("i2s", blob, 64, 1024, [24, 64], [1.0, 1.0], x)      # 24 is not a multiple of 16
    with pytest.raises(bn.BitnetError, match="invalid"):
        bn.bitnet_linear_segments("i2s", blob, 64, 1024, [32, 48], [1.0, 1.0], x)      # does not end at M
    with pytest.raises(bn.BitnetError, match="invalid"):
        bn.bitnet_linear_segments("i2s", blob, 64, 1024, [32, 32, 64], [1.0, 1.0, 1.0], x)   # empty segment


def test_group_tl2_long_rows_walked_in_parts():
    """TL2 batches whose staged codes do not fit beside the decode table: the triple tiles of a row are walked in
    parts, the pair tiles of the tail with the last part, the integer sums resting in y in between."""
    shapes = [(64, 14336, 8), (96, 28672, 4), (32, 28672, 8), (160, 96 * 150 + 92, 7), (64, 8192, 8), (320, 28672, 2),
              (32, 96 * 9, 1)]
    items = [Item("tl2", M, K, T, 1200 + i) for i, (M, K, T) in enumerate(shapes)]
    run_group(items)
    for it in items:
        it.check()
    run_group(items)            # y held integer scratch in between: nothing stale may survive
    for it in items:
        it.check()

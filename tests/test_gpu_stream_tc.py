"""17 to 128 tokens per linear through the list call: the streaming tensor-core kernel (weights read once, unpacked
into tensor memory, tcgen05 MMAs with unsigned codes, sum(q) taken off in the epilogue) against the CPU oracle."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth
from test_gpu_group import Item, run_group

pytestmark = pytest.mark.gpu


def test_stream_tc_one_small_item():
    items = [Item("i2s", 128, 2048, 17, 800)]
    run_group(items)
    items[0].check()


def test_stream_tc_ragged_rows_token_counts_and_long_rows():
    """Rows that are no multiple of the 128-row tile, K with a padded last chunk (K % 256 = 64), 17..64 tokens, a
    28672-column row, neighbours the other grouped kernels take (1 and 12 tokens) in the same list."""
    shapes = [(300, 4096, 24), (1000, 8192, 64), (64, 28672, 33), (5, 2112, 40), (129, 3200, 17), (160, 8192, 1),
              (96, 4096, 12), (2048, 2048, 63)]
    items = [Item("i2s", M, K, T, 810 + i) for i, (M, K, T) in enumerate(shapes)]
    run_group(items)
    for it in items:
        it.check()


def test_stream_tc_many_tiles_per_cta_and_repeat():
    """More tiles than CTAs (every CTA walks several tiles and both accumulators), run twice in a row."""
    items = [Item("i2s", 24576, 2048, 32, 830), Item("i2s", 8192, 4096, 48, 831)]
    rng = np.random.default_rng(3)
    for _ in range(2):
        run_group(items)
        for it in items:
            it.check(rows=np.sort(rng.choice(it.M, 300, replace=False)))


def test_stream_tc_more_items_than_one_launch_takes():
    """More items than one argument block holds (160: a tensor map per item): several launches in list order; every
    CTA meets several items (the per-token sums are taken anew at each), K with an odd number of 256-column chunks."""
    items = [Item("i2s", 128 * (1 + i % 2) - (i % 5), 2048 + 256 * (i % 4), 17 + i % 20, 3500 + i) for i in range(170)]
    run_group(items)
    for it in items:
        it.check()


def test_stream_tc_same_list_ten_times():
    """One tile per CTA, cold and warm: the packed-word ring must not be refilled before every warp has used its
    words, whatever the timing (ten runs, every accumulator each time)."""
    it = Item("i2s", 1000, 8192, 64, 811)
    q_ref, _, _ = oracle.quant_act(it.x.numpy())
    acc_ref = oracle.mpgemm_def(q_ref, it.w.numpy())
    for _ in range(10):
        it.gacc.t.zero_()
        run_group([it])
        assert np.array_equal(it.gacc.t.cpu().numpy(), acc_ref)


def test_stream_tc_leaves_very_long_rows_to_other_kernels():
    """K beyond 131072 (64 x the sums would leave 32 bits) is not taken by the streaming kernel: the list call hands
    such items to the single-call kernels, K = 131072 itself still runs here; both agree with the oracle."""
    items = [Item("i2s", 96, 131072, 20, 890), Item("i2s", 64, 131072 + 64, 20, 891)]
    run_group(items)
    for it in items:
        it.check()


def test_stream_tc_sixty_five_to_128_tokens():
    """The 128-token tile variant (two activation pieces per writer thread and K block, 8 stages), mixed with
    64-token items in one list (separate launches per class), ragged rows and a long row."""
    shapes = [(128, 2048, 65), (300, 4096, 100), (1000, 8192, 128), (64, 28672, 77), (129, 3200, 33), (2048, 2048, 127),
              (96, 4096, 128)]
    items = [Item("i2s", M, K, T, 850 + i) for i, (M, K, T) in enumerate(shapes)]
    run_group(items)
    for it in items:
        it.check()


def test_stream_tc_serves_large_single_calls():
    """bitnet_mpgemm / bitnet_linear on one tensor with many 128-row tiles and 33 to 128 tokens take the same kernel
    (sampled rows against the oracle); the same call with the switch off must give identical bits."""
    from helpers import check_y, npy
    for M, K, T in [(14336, 4096, 48), (40000, 2048, 100)]:
        w = synth.ternary(870, 1, M, K, 1 / 3, 1 / 3)
        x = synth.normal(871, T, T, K)
        blob = bn.pack("i2s", w.cuda())
        y, q, sc, acc = bn.bitnet_linear("i2s", blob, 0.5, M, K, x.cuda(), want_acc=True)
        torch.cuda.synchronize()
        rows = np.sort(np.random.default_rng(7).choice(M, 400, replace=False))
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(q), q_ref)
        acc_ref = oracle.mpgemm_def(q_ref, np.ascontiguousarray(w.numpy()[rows]))
        assert np.array_equal(npy(acc)[:, rows], acc_ref)
        check_y(y[:, torch.as_tensor(rows).cuda()], acc_ref, sc_ref, 0.5)
    assert bn.bitnet_device_status() == 0

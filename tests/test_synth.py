"""The seeded input generators: determinism, row re-draws, the weight law and the outlier recipe."""
import numpy as np
import torch

from paper_2502_11880_b200 import synth


def test_mix64_tensor_matches_python_ints():
    u = synth.draw_u64(7, 3, 5, 4)
    key = synth.stream_key(7, 3)
    for i in range(4):
        assert (int(u[i]) & ((1 << 64) - 1)) == synth._mix64_int((key + 5 + i) & ((1 << 64) - 1))


def test_ternary_law_and_row_redraw():
    w = synth.ternary(2, 1, 64, 4096, 0.4, 0.3)
    assert set(np.unique(w.numpy()).tolist()) == {-1, 0, 1}
    frac0 = float((w == 0).float().mean())
    fracp = float((w == 1).float().mean())
    assert abs(frac0 - 0.4) < 0.01 and abs(fracp - 0.3) < 0.01
    again = synth.ternary(2, 1, 5, 4096, 0.4, 0.3, row_start=17)
    assert torch.equal(again, w[17:22])
    chunked = synth.ternary(2, 1, 64, 4096, 0.4, 0.3, chunk_elems=1000)
    assert torch.equal(chunked, w)


def test_normal_moments_and_outliers():
    x = synth.normal(0, 4, 2, 20000)
    assert abs(float(x.mean())) < 0.02 and abs(float(x.std()) - 1.0) < 0.02
    wl = synth.CONFIGS["gemv1536"]
    a = wl.activations(0, 0, 1)
    assert a.shape == (1, 1536)
    assert int((a.abs() == 20.0).sum()) == 2          # ceil(0.001 * 1536)
    assert torch.equal(a, wl.activations(0, 0, 1))


def test_workload_shapes():
    s = synth.CONFIGS["sweep100b"]
    per_layer = sum(l.K * l.M for l in s.linears)
    assert per_layer == 8192 * 10240 + 8192 * 8192 + 8192 * 57344 + 28672 * 8192
    assert s.layers * per_layer // 4 == 17112760320        # I2_S bytes of the whole sweep
    w = s.weights(3, 1, rows=2, row_start=8190)
    assert w.shape == (2, 8192)
    assert abs(synth.absmean_scale(synth.ternary(1, 0, 32, 3200, 1 / 3, 1 / 3)) - 2 / 3) < 0.01

"""GPU parity: every step of the CUDA path against the CPU oracle, through the C ABI, on the same
seeded inputs.  Integers, bytes and scale bit patterns must be identical; fp32 outputs within 1e-6
relative."""
import numpy as np
import pytest
import torch

import oracle
import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth

from helpers import check_linear, check_y, dev, no_workspace, npy, oracle_pack, run_fused, run_linear

pytestmark = pytest.mark.gpu


def tern(seed, M, K, p0=1 / 3, pp=1 / 3):
    return synth.ternary(seed, 99, M, K, p0, pp)


# ----------------------------------------------------------------------------- quantiser
@pytest.mark.parametrize("T,K", [(1, 1), (1, 7), (3, 64), (2, 1536), (1, 28672), (8, 4096), (5, 1001), (64, 333),
                                 (5, 8192), (8, 16384), (4, 32768), (7, 8200), (6, 16388), (9, 8192), (3, 16384)])   # 4-8 tokens: clusters of 4 / 8 CTAs per row
def test_quant_bit_exact(T, K):
    x = synth.normal(11, T * 1000 + K % 997, T, K)
    q, sc, sm = bn.bitnet_quant_act(x.cuda())
    q_ref, sc_ref, sm_ref = oracle.quant_act(x.numpy())
    assert np.array_equal(npy(q), q_ref)
    assert np.array_equal(npy(sc).view(np.uint32), sc_ref.view(np.uint32))
    assert np.array_equal(npy(sm), sm_ref)


def test_quant_ties_zero_rows_outliers_per_tensor():
    x = torch.zeros(4, 128)
    x[0, :9] = torch.tensor([127.0, 0.5, 1.5, 2.5, -0.5, -1.5, 126.5, -2.5, 3.5])
    x[2] = synth.add_outliers(synth.normal(1, 2, 1, 128), 1, 2, 0.02)[0]
    x[3] = 1e-7 * synth.normal(1, 3, 1, 128)[0]         # below the 1e-5 floor
    for per_tensor in (False, True):
        q, sc, sm = bn.bitnet_quant_act(x.cuda(), per_tensor=per_tensor)
        q_ref, sc_ref, sm_ref = oracle.quant_act(x.numpy(), per_tensor=per_tensor)
        assert np.array_equal(npy(q), q_ref)
        assert np.array_equal(npy(sc).view(np.uint32), sc_ref.view(np.uint32))
        assert np.array_equal(npy(sm), sm_ref)
    assert npy(q)[1].any() == False  # noqa: E712  (all-zero row stays zero)


# ----------------------------------------------------------------------------- packers
@pytest.mark.parametrize("M,K", [(1, 64), (5, 128), (33, 192), (100, 8640), (7, 1536)])
def test_pack_i2s_bytes_and_round_trip(M, K):
    w = tern(3, M, K)
    blob = bn.bitnet_pack_i2s(w.cuda())
    assert np.array_equal(npy(blob), oracle.pack_i2s(w.numpy()))
    assert torch.equal(bn.bitnet_unpack_i2s(blob, M, K).cpu(), w)
    # the GPU inverse also decodes the oracle's blob
    assert torch.equal(bn.bitnet_unpack_i2s(dev(oracle.pack_i2s(w.numpy())), M, K).cpu(), w)


@pytest.mark.parametrize("fmt,M,K,bk3", [("tl1", 32, 2, 0), ("tl1", 64, 130, 0), ("tl2", 32, 96, 0),
                                         ("tl2", 96, 3200, 0), ("tl2", 64, 8640, 0), ("tl2", 32, 4096, 0),
                                         ("tl2", 64, 1000, 192), ("tl2", 32, 34, 0)])
def test_pack_tl_bytes_and_round_trip(fmt, M, K, bk3):
    w = tern(4, M, K, 0.4, 0.3)
    blob = bn.bitnet_pack_tl(fmt, w.cuda(), bk3)
    assert np.array_equal(npy(blob), oracle.pack_tl(fmt, w.numpy(), bk3))
    assert torch.equal(bn.bitnet_unpack_tl(fmt, blob, M, K, bk3).cpu(), w)


def test_packers_flag_non_ternary_input():
    w = tern(5, 32, 192)
    w[3, 17] = 2
    for f in (lambda: bn.bitnet_pack_i2s(w.cuda()), lambda: bn.bitnet_pack_tl("tl2", w.cuda()),
              lambda: bn.bitnet_pack_tl("tl1", w.cuda())):
        with pytest.raises(bn.BitnetError, match="weight"):
            f()


@pytest.mark.parametrize("fmt,K", [("tl2", 96 * 3 + 64), ("tl2", 3200), ("tl1", 130)])
def test_tl_tables_match_precompute(fmt, K):
    q = torch.randint(-127, 128, (K,), dtype=torch.int8, generator=torch.Generator().manual_seed(K))
    lut = bn.bitnet_tl_build_lut_debug(fmt, q.cuda())
    assert np.array_equal(npy(lut), oracle.tl_build_lut(fmt, q.numpy()))


# ----------------------------------------------------------------------------- mpGEMV, small and ragged shapes
SHAPES = [(32, 64), (64, 128), (96, 3200), (160, 8640), (32, 2048 * 5 + 64), (224, 1536), (32, 4096 + 2048)]


@pytest.mark.parametrize("fmt", ["i2s", "tl1", "tl2"])
@pytest.mark.parametrize("T", [1, 2, 3, 5, 8])
def test_mpgemv_parity(fmt, T):
    for i, (M, K) in enumerate(SHAPES):
        w = tern(20 + i, M, K, 0.4, 0.3)
        x = synth.normal(21, i * 16 + T, T, K)
        check_linear(fmt, w, x)


@pytest.mark.parametrize("fmt", ["i2s", "tl2"])
@pytest.mark.parametrize("T", [1, 2, 3, 8, 11])
def test_linear_from_fp32_matches_oracle(fmt, T):
    """bitnet_linear (one fused kernel for I2_S decode, two kernels otherwise) against the oracle."""
    for i, (M, K) in enumerate([(64, 128), (96, 3200), (160, 8640), (32, 28672), (224, 8192), (32, 1536)]):
        w = tern(70 + i, M, K)
        x = synth.normal(71, i * 16 + T, T, K)
        blob = bn.pack(fmt, w.cuda())
        y, q, sc, acc = run_fused(fmt, blob, 0.75, M, K, x.cuda())
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(q), q_ref)
        assert np.array_equal(npy(sc).view(np.uint32), sc_ref.view(np.uint32))
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(acc), acc_ref)
        check_y(y, acc_ref, sc_ref, 0.75)


def test_i2s_rows_not_multiple_of_anything():
    for M in (1, 7, 9, 300):
        check_linear("i2s", tern(30, M, 256), synth.normal(30, M, 2, 256))


@pytest.mark.parametrize("fmt", ["i2s", "tl1", "tl2"])
def test_constant_weights_and_workspace_reuse(fmt):
    M, K, T = 64, 28672, 2            # long K: several K-slices meet in the workspace
    x = synth.normal(31, 1, T, K)
    q_ref, sc_ref, sm_ref = oracle.quant_act(x.numpy())
    ws = bn.new_workspace(fmt, T, M, K)
    assert ws is not None or fmt == "i2s"      # the I2_S kernel joins its K-slices inside the CTA
    for val in (0, 1, -1, 1):          # the same workspace serves every call: it must come back clean
        w = torch.full((M, K), val, dtype=torch.int8)
        out = run_linear(fmt, w, x, workspace=ws, w_scale=0.5)
        expect = np.repeat((val * sm_ref.astype(np.int64))[:, None], M, axis=1).astype(np.int32)
        assert np.array_equal(npy(out["acc"]), expect)
        check_y(out["y"], expect, sc_ref, 0.5)
    # the head of the workspace (split-K sums and arrival counters) must come back zeroed
    assert ws is None or not npy(ws)[: (T * M + M) * 4].any()


def test_i2s_streaming_kernel_edges():
    """Shapes that stress the warp-ring decode kernel: fewer rows than one 16-row unit, ragged last unit,
    K exactly one ring long (2048), six tokens, and more units per CTA than the fixed first two per warp
    group (20000 rows at K = 8192), each with given codes and fused.  Offered a workspace, the crowded
    batches (six tokens; five and four at K = 28672) go to the mid-batch kernel instead: both must agree."""
    shapes = [(1, 4096, 1), (17, 4096, 3), (300, 2048, 6), (33, 2048, 1), (48, 28672, 5), (48, 28672, 4),
              (20000, 8192, 4)]
    for (M, K, T) in shapes:
        w, x = tern(36, M, K), synth.normal(36, M + T, T, K)
        out = check_linear("i2s", w, x, workspace=no_workspace())     # given codes, decode kernel
        y, q, sc, acc = run_fused("i2s", out["blob"], out["w_scale"], M, K, x.cuda(), workspace=no_workspace())   # fused
        assert torch.equal(acc, out["acc"]) and torch.equal(y, out["y"]) and torch.equal(q, out["q"])
        y, q, sc, acc = run_fused("i2s", out["blob"], out["w_scale"], M, K, x.cuda())
        # (with whatever workspace the shape asks for)
        assert torch.equal(acc, out["acc"]) and torch.equal(y, out["y"]) and torch.equal(q, out["q"])
        if bn.bitnet_mpgemm_workspace_bytes("i2s", T, M, K):
            assert (T >= 6 or T * K > 96 * 1024)
            check_linear("i2s", w, x)                                 # given codes, mid-batch kernel


def test_i2s_very_long_k_runs_in_phases():
    M, K = 48, 1 << 17
    for T in (1, 2):
        check_linear("i2s", tern(34, M, K), synth.normal(34, T, T, K))


def test_tl_many_row_blocks_few_tiles():
    # more row blocks per CTA than the kernel keeps cross-warp sums for, and fewer tiles than warps
    M, K = 32 * 296 * 70, 96
    w, x = tern(35, M, K), synth.normal(35, 1, 2, K)
    for fmt in ("tl2", "tl1"):
        out = run_linear(fmt, w, x)
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(out["acc"]), oracle.mpgemm_def(q_ref, w.numpy()))


def test_i2s_mid_batch_kernel_every_tile_count():
    """9 to 64 tokens (the mma.sync weight scan over K-slices): every number of 8-token tiles, ragged last
    tiles, odd numbers of 16-row units, K that needs padding, one and many K-slices."""
    shapes = [(7, 1024), (33, 3200), (300, 8640), (200, 28672), (2000, 2048)]
    for i, (M, K) in enumerate(shapes):
        w = tern(40 + i, M, K, 0.4, 0.3)
        for T in (9, 16, 17, 24, 25, 32, 33, 40, 41, 48, 49, 56, 57, 64):
            if M * K * T > 400e6 and T not in (9, 32, 57, 64):
                continue                      # keep the oracle's share of the test to seconds
            assert bn.bitnet_mpgemm_workspace_bytes("i2s", T, M, K) >= T * M * 4
            check_linear("i2s", w, synth.normal(41, i * 100 + T, T, K))


def test_i2s_mid_batch_workspace_comes_back_clean_and_is_optional():
    M, K, T = 96, 8192, 40
    w, x = tern(42, M, K), synth.normal(42, 1, T, K)
    ws = bn.new_workspace("i2s", T, M, K)
    first = run_linear("i2s", w, x, workspace=ws)
    assert not npy(ws).any()
    again = run_linear("i2s", w, x, workspace=ws)        # the sums of the first call are gone
    assert torch.equal(first["acc"], again["acc"]) and torch.equal(first["y"], again["y"])
    acc_ref = oracle.mpgemm_def(oracle.quant_act(x.numpy())[0], w.numpy())
    assert np.array_equal(npy(again["acc"]), acc_ref)
    # without a workspace the call still succeeds (the tensor-core prefill kernel takes it): same numbers
    y2 = torch.empty_like(first["y"])
    acc2 = torch.empty_like(first["acc"])
    rc = bn.lib().bitnet_mpgemm(0, first["blob"].data_ptr(), first["w_scale"], M, K, 0, first["q"].data_ptr(),
                                first["act_scale"].data_ptr(), T, y2.data_ptr(), acc2.data_ptr(), None, 0, None)
    torch.cuda.synchronize()
    assert rc == 0
    assert torch.equal(acc2, first["acc"]) and torch.equal(y2, first["y"])


def test_i2s_mid_batch_in_a_graph_with_early_start():
    """Quantiser, scan and rescale kernels of several linears back to back in one CUDA graph (programmatic
    dependent launch between them), sharing one workspace: the benchmark-style launch configuration."""
    T = 24
    shapes = [(512, 4096), (4096, 2048), (640, 8192)]
    ws_bytes = max(bn.bitnet_mpgemm_workspace_bytes("i2s", T, M, K) for M, K in shapes)
    ws = torch.zeros(ws_bytes, dtype=torch.uint8, device="cuda")
    items = []
    for i, (M, K) in enumerate(shapes):
        w, x = tern(43 + i, M, K), synth.normal(43, i, T, K)
        items.append(dict(M=M, K=K, w=w, x=x.cuda(), blob=bn.pack("i2s", w.cuda()),
                          q=torch.empty((T, K), dtype=torch.int8, device="cuda"),
                          sc=torch.empty(T, dtype=torch.float32, device="cuda"),
                          y=torch.empty((T, M), dtype=torch.float32, device="cuda"),
                          acc=torch.empty((T, M), dtype=torch.int32, device="cuda")))

    def run():
        for d in items:
            bn.bitnet_linear("i2s", d["blob"], 0.5, d["M"], d["K"], d["x"], q=d["q"], act_scale=d["sc"], y=d["y"],
                             acc_out=d["acc"], workspace=ws)
    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        run()
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        run()
    for d in items:
        d["y"].zero_(), d["acc"].zero_()
    for _ in range(3):
        g.replay()
    torch.cuda.synchronize()
    for d in items:
        q_ref, sc_ref, _ = oracle.quant_act(d["x"].cpu().numpy())
        acc_ref = oracle.mpgemm_def(q_ref, d["w"].numpy())
        assert np.array_equal(npy(d["acc"]), acc_ref)
        check_y(d["y"], acc_ref, sc_ref, 0.5)
    assert not npy(ws).any()


def test_formats_agree_on_accumulators():
    M, K, T = 128, 8192, 3
    w, x = tern(32, M, K), synth.normal(32, 1, T, K)
    accs = [npy(run_linear(f, w, x)["acc"]) for f in ("i2s", "tl1", "tl2")]
    assert np.array_equal(accs[0], accs[1]) and np.array_equal(accs[0], accs[2])


def test_many_tokens_tl_and_i2s():
    M, K, T = 64, 1536, 21            # more than 8 tokens
    w, x = tern(33, M, K), synth.normal(33, 1, T, K)
    for fmt in ("tl2", "i2s"):
        check_linear(fmt, w, x)


# ----------------------------------------------------------------------------- the five workloads
def test_workload_gemv1536_all_formats():
    wl = synth.CONFIGS["gemv1536"]
    w, x = wl.weights(0, 0), wl.activations(0, 0, 1)
    for fmt in wl.formats:
        check_linear(fmt, w, x)


@pytest.mark.parametrize("name", ["layer3b", "layer8b"])
def test_workload_layers_full_parity(name):
    wl = synth.CONFIGS[name]
    for j, lin in enumerate(wl.linears):
        w = wl.weights(0, j)
        for T in wl.tokens:
            x = wl.activations(0, j, T)
            for fmt in wl.formats:
                check_linear(fmt, w, x)


def _sampled_rows(M, n=96, seed=0):
    g = np.random.default_rng(seed)
    rows = np.unique(np.concatenate([[0, 1, 31, 32, M - 33, M - 32, M - 1], g.integers(0, M, n)]))
    return rows


@pytest.mark.parametrize("layer", [0, 79])
def test_workload_sweep100b_sampled_rows(layer):
    """Full-size tensors of the 100B-shaped sweep, built and packed in device memory exactly as the
    benchmark does; the oracle recomputes sampled output rows from host re-draws of the same weights."""
    wl = synth.CONFIGS["sweep100b"]
    for j, lin in enumerate(wl.linears):
        wd = wl.weights(layer, j, device="cuda")
        x = wl.activations(layer, j, 1)
        q, sc, sm = bn.bitnet_quant_act(x.cuda())
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        assert np.array_equal(npy(q), q_ref)
        rows = _sampled_rows(lin.M, seed=layer * 4 + j)
        w_rows = np.stack([wl.weights(layer, j, row_start=int(r), rows=1).numpy()[0] for r in rows])
        assert np.array_equal(npy(wd[torch.as_tensor(rows).cuda()]), w_rows)
        acc_ref = oracle.mpgemm_def(q_ref, w_rows)
        w_scale = 2.0 / 3.0
        for fmt in wl.formats:
            blob = bn.pack(fmt, wd, check=False)
            y, acc = bn.bitnet_mpgemm(fmt, blob, w_scale, lin.M, lin.K, q, sc, want_acc=True)
            torch.cuda.synchronize()
            assert np.array_equal(npy(acc)[:, rows], acc_ref)
            check_y(y[:, torch.as_tensor(rows).cuda()], acc_ref, sc_ref, w_scale)
            # whole-vector properties: TL and I2_S agree everywhere; accumulators bounded by 127*K
            if fmt == "i2s":
                acc_i2s = acc.clone()
            else:
                assert torch.equal(acc, acc_i2s)
            assert int(acc.abs().max()) <= 127 * lin.K
            del blob
        del wd
        torch.cuda.empty_cache()


def test_sweep100b_layer_in_the_benchmark_launch_configuration():
    """One full-size layer of the sweep exactly as bench.py runs it: the four linears as fused bitnet_linear
    calls (fp32 activations in), captured in a CUDA graph with programmatic dependent launch and replayed;
    sampled output rows against the oracle, twice (the second replay must not depend on the first)."""
    wl = synth.CONFIGS["sweep100b"]
    layer = 3
    blobs, xs, ys, qs, scs, rows_l, refs = [], [], [], [], [], [], []
    w_scale = 2.0 / 3.0
    for j, lin in enumerate(wl.linears):
        wd = wl.weights(layer, j, device="cuda")
        blobs.append(bn.pack("i2s", wd, check=False))
        del wd
        x = wl.activations(layer, j, 1)
        xs.append(x.cuda())
        ys.append(torch.zeros((1, lin.M), dtype=torch.float32, device="cuda"))
        qs.append(torch.empty((1, lin.K), dtype=torch.int8, device="cuda"))
        scs.append(torch.empty(1, dtype=torch.float32, device="cuda"))
        rows = _sampled_rows(lin.M, seed=100 + j)
        w_rows = np.stack([wl.weights(layer, j, row_start=int(r), rows=1).numpy()[0] for r in rows])
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        rows_l.append(rows)
        refs.append((q_ref, sc_ref, oracle.mpgemm_def(q_ref, w_rows)))
    ws = torch.zeros(64, dtype=torch.uint8, device="cuda")

    def layer_step():
        for j, lin in enumerate(wl.linears):
            bn.bitnet_linear("i2s", blobs[j], w_scale, lin.M, lin.K, xs[j], q=qs[j], act_scale=scs[j], y=ys[j], workspace=ws)

    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        layer_step()
    torch.cuda.current_stream().wait_stream(s)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g):
        layer_step()
    for rep in range(2):
        for y in ys:
            y.zero_()
        g.replay()
        torch.cuda.synchronize()
        for j in range(len(wl.linears)):
            q_ref, sc_ref, acc_ref = refs[j]
            assert np.array_equal(npy(qs[j]), q_ref), (rep, j)
            assert np.array_equal(npy(scs[j]).view(np.uint32), sc_ref.view(np.uint32)), (rep, j)
            check_y(ys[j][:, torch.as_tensor(rows_l[j]).cuda()], acc_ref, sc_ref, w_scale)
    assert bn.bitnet_device_status() == 0


def test_prefill_output_paths_agree():
    """The prefill kernel writes y either with plain stores (when the accumulators are asked for, or M % 4 != 0)
    or through shared memory and bulk tensor stores: same bits, nothing written outside y, ragged M and T."""
    for (M, K, T) in [(300, 1024, 70), (128, 512, 256), (1000, 2048, 333), (130, 512, 65)]:
        w, x = tern(50, M, K), synth.normal(50, M + T, T, K)
        out = check_linear("i2s", w, x)                       # with accumulators: plain stores, against the oracle
        guard = torch.full((T + 8, M), 12345.0, dtype=torch.float32, device="cuda")
        y = guard[4: T + 4]                                   # four rows in: 16-byte aligned for every M
        bn.bitnet_mpgemm("i2s", out["blob"], out["w_scale"], M, K, out["q"], out["act_scale"], y=y)
        torch.cuda.synchronize()
        assert torch.equal(y, out["y"])
        assert bool((guard[:4] == 12345.0).all()) and bool((guard[T + 4:] == 12345.0).all())


def test_prefill_few_tiles_split_k():
    """More than 64 tokens on a layer with fewer output tiles than SMs: every tile's K is cut into parts that
    meet in the workspace (integer atomics) and a second kernel rescales; long K, ragged M and T, and the same
    call without a workspace (whole tiles) must agree."""
    for (M, K, T) in [(300, 8192, 70), (1000, 28672, 130), (130, 4096, 65)]:
        w, x = tern(52, M, K), synth.normal(52, M + T, T, K)
        assert bn.bitnet_mpgemm_workspace_bytes("i2s", T, M, K) >= T * M * 4
        ws = bn.new_workspace("i2s", T, M, K)
        out = check_linear("i2s", w, x, workspace=ws)
        assert not npy(ws).any()
        again = run_linear("i2s", w, x, workspace=ws)
        assert torch.equal(again["acc"], out["acc"]) and torch.equal(again["y"], out["y"])
        whole = run_linear("i2s", w, x, workspace=no_workspace())
        assert torch.equal(whole["acc"], out["acc"]) and torch.equal(whole["y"], out["y"])


def test_workload_prefill_sampled():
    wl = synth.CONFIGS["prefill"]
    lin = wl.linears[0]
    T = wl.tokens[0]
    w, x = wl.weights(0, 0), wl.activations(0, 0, T)
    out = run_linear("i2s", w, x)
    q_ref, sc_ref, sm_ref = oracle.quant_act(x.numpy())
    assert np.array_equal(npy(out["q"]), q_ref)
    assert np.array_equal(npy(out["act_scale"]).view(np.uint32), sc_ref.view(np.uint32))
    rows = _sampled_rows(lin.M, 64, seed=3)
    toks = np.unique(np.concatenate([[0, 1, 127, 128, T - 1], np.random.default_rng(3).integers(0, T, 40)]))
    acc_ref = oracle.mpgemm_def(q_ref[toks], w.numpy()[rows])
    acc = npy(out["acc"])[np.ix_(toks, rows)]
    assert np.array_equal(acc, acc_ref)
    check_y(out["y"][torch.as_tensor(toks).cuda()][:, torch.as_tensor(rows).cuda()], acc_ref, sc_ref[toks],
            out["w_scale"])
    # all-ones weights: every output of a token equals that token's code sum (a whole-matrix property)
    ones = torch.ones(256, lin.K, dtype=torch.int8)
    o2 = run_linear("i2s", ones, x, w_scale=1.0)
    assert torch.equal(o2["acc"], o2["act_sum"][:, None].expand(T, 256).contiguous())


# ----------------------------------------------------------------------------- kernel variants and device status
def test_early_start_off_gives_the_same_results():
    M, K, T = 96, 8192, 2
    w, x = tern(50, M, K), synth.normal(50, 1, T, K)
    a = run_linear("i2s", w, x)
    bn.bitnet_set_early_start(False)
    try:
        b = run_linear("i2s", w, x)
    finally:
        bn.bitnet_set_early_start(True)
    assert torch.equal(a["acc"], b["acc"]) and torch.equal(a["y"], b["y"]) and torch.equal(a["q"], b["q"])


def test_back_to_back_launches_keep_stream_order():
    # quantiser -> GEMV chains queued without any host synchronisation, different inputs every round
    M, K = 512, 8192
    w = tern(51, M, K)
    blob = bn.pack("i2s", w.cuda())
    xs = [synth.normal(51, 10 + i, 1, K) for i in range(6)]
    xd = [x.cuda() for x in xs]
    q = torch.empty((1, K), dtype=torch.int8, device="cuda")
    sc = torch.empty(1, dtype=torch.float32, device="cuda")
    sm = torch.empty(1, dtype=torch.int32, device="cuda")
    ys = [torch.empty((1, M), dtype=torch.float32, device="cuda") for _ in xs]
    accs = [torch.empty((1, M), dtype=torch.int32, device="cuda") for _ in xs]
    torch.cuda.synchronize()
    for fused in (False, True):
        for i in range(len(xs)):           # the same q / scale buffers are rewritten every round
            if fused:
                bn.bitnet_linear("i2s", blob, 1.0, M, K, xd[i], q=q, act_scale=sc, y=ys[i], acc_out=accs[i])
            else:
                bn.bitnet_quant_act(xd[i], q=q, act_scale=sc, act_sum=sm)
                bn.bitnet_mpgemm("i2s", blob, 1.0, M, K, q, sc, y=ys[i], acc_out=accs[i])
        torch.cuda.synchronize()
        for i, x in enumerate(xs):
            q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
            acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
            assert np.array_equal(npy(accs[i]), acc_ref), (fused, i)
            check_y(ys[i], acc_ref, sc_ref, 1.0)
            ys[i].zero_()
            accs[i].zero_()


def test_split_k_kernel_variant_in_a_child_process():
    # BITNET_I2S_KERNEL=splitk selects the register-resident split-K kernel (read once per process)
    import os
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, 'tests'); import numpy as np, torch\n"
        "from paper_2502_11880_b200 import synth\n"
        "from helpers import check_linear\n"
        "for T in (1, 2, 5):\n"
        "    for (M, K) in [(40, 1536), (64, 28672), (33, 8640)]:\n"
        "        check_linear('i2s', synth.ternary(60, 1, M, K, 1/3, 1/3), synth.normal(60, T, T, K))\n"
        "print('ok')\n")
    env = dict(os.environ, BITNET_I2S_KERNEL="splitk")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert out.returncode == 0 and "ok" in out.stdout, out.stderr[-2000:]


def test_prefill_forced_split_and_mid_batch_off_in_child_processes():
    """Read-once switches: BITNET_PREFILL_KSPLIT forces the number of K parts per tile (here 3 and 8, on shapes
    with several tiles per SM round and a ragged last part), BITNET_I2S_MID_MAX_T=0 sends 9 to 64 tokens to the
    prefill kernel.  Each must still agree with the oracle."""
    import os
    import subprocess
    import sys
    code = (
        "import sys; sys.path.insert(0, 'tests'); import numpy as np, torch\n"
        "from paper_2502_11880_b200 import synth\n"
        "import paper_2502_11880_b200 as bn\n"
        "from helpers import check_linear\n"
        "for (M, K, T) in [(700, 5120, 70), (130, 28672, 300), (2000, 2048, 33), (64, 8192, 12)]:\n"
        "    check_linear('i2s', synth.ternary(61, 1, M, K, 1/3, 1/3), synth.normal(61, T, T, K))\n"
        "assert bn.bitnet_device_status() == 0\n"
        "print('ok')\n")
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    for extra in (dict(BITNET_PREFILL_KSPLIT="3"), dict(BITNET_PREFILL_KSPLIT="8"), dict(BITNET_I2S_MID_MAX_T="0")):
        env = dict(os.environ, **extra)
        out = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
        assert out.returncode == 0 and "ok" in out.stdout, (extra, out.stderr[-2000:])


def test_zzz_no_device_wait_ever_gave_up():
    assert bn.bitnet_device_status() == 0


@pytest.mark.gpu
def test_linear_host_batch_matches_single_calls():
    """bitnet_linear_host_batch (overlapped copies) gives what bitnet_linear gives item by item, for a mix
    of formats, shapes and batch sizes, and leaves the stream joined (two batches back to back)."""
    shapes = [("i2s", 512, 2048, 1), ("i2s", 96, 8192, 2), ("tl2", 64, 1536, 1), ("i2s", 1040, 4096, 4), ("tl1", 128, 256, 3)]
    items, keep, refs, orc = [], [], [], []
    for n, (fmt, M, K, T) in enumerate(shapes):
        w = synth.ternary(40 + n, 0, M, K, 1 / 3, 1 / 3)
        x = synth.normal(40 + n, 1, T, K)
        blob = bn.pack(fmt, w.cuda())
        xh = x.clone().pin_memory()
        yh = torch.zeros((T, M), dtype=torch.float32).pin_memory()
        xd = torch.empty((T, K), dtype=torch.float32, device="cuda")
        qd = torch.empty((T, K), dtype=torch.int8, device="cuda")
        sd = torch.empty(T, dtype=torch.float32, device="cuda")
        yd = torch.empty((T, M), dtype=torch.float32, device="cuda")
        ws = bn.new_workspace(fmt, T, M, K)
        items.append(dict(fmt=fmt, packed=blob, w_scale=0.75, M=M, K=K, x_host=xh, y_host=yh, x_dev=xd, q_dev=qd,
                          scale_dev=sd, y_dev=yd, workspace=ws))
        keep.append((blob, xh, yh, xd, qd, sd, yd, ws))
        q = torch.empty_like(qd)
        sc = torch.empty_like(sd)
        y = torch.empty_like(yd)
        bn.bitnet_linear(fmt, blob, 0.75, M, K, x.cuda(), q=q, act_scale=sc, y=y, workspace=bn.new_workspace(fmt, T, M, K))
        refs.append(y.cpu())
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        orc.append((q_ref, sc_ref, oracle.mpgemm_def(q_ref, w.numpy())))
    batch = bn.make_host_batch(items)
    for rep in range(2):
        for it in items:
            it["y_host"].zero_()
        bn.bitnet_linear_host_batch(batch)
        torch.cuda.current_stream().synchronize()
        for n, (it, ref) in enumerate(zip(items, refs)):
            assert torch.equal(it["y_host"], ref), (rep, it["fmt"], it["M"], it["K"])
            # and directly against the oracle: the host result, and the codes and scales left on the device
            q_ref, sc_ref, acc_ref = orc[n]
            check_y(it["y_host"], acc_ref, sc_ref, 0.75)
            assert np.array_equal(npy(it["q_dev"]), q_ref)
            assert np.array_equal(npy(it["scale_dev"]).view(np.uint32), sc_ref.view(np.uint32))
    assert bn.bitnet_device_status() == 0


@pytest.mark.gpu
def test_linear_host_batch_merges_neighbouring_buffers():
    """Items whose host and device buffers continue one another (one pinned block, one device block) travel as
    one copy per group (40 items: five groups, the copies of one under the kernels of its
    neighbour); items 3 and 4 break the chain on the host side only, the last item has 24 tokens (streaming or
    mid-batch kernel).  Same results as item-by-item calls, nothing outside the buffers touched."""
    specs = [(256, 1024, 1)] * 3 + [(512, 2048, 2)] * 36 + [(320, 4096, 24)]
    nx = sum(T * K for M, K, T in specs)
    ny = sum(T * M for M, K, T in specs)
    xh_all = torch.empty(nx + 64, dtype=torch.float32).pin_memory()
    yh_all = torch.full((ny + 64,), -7.0, dtype=torch.float32).pin_memory()
    xd_all = torch.empty(nx, dtype=torch.float32, device="cuda")
    yd_all = torch.empty(ny, dtype=torch.float32, device="cuda")
    items, refs, keep = [], [], []
    xo = xd_o = yo = 0
    for n, (M, K, T) in enumerate(specs):
        w = synth.ternary(60 + n, 0, M, K, 1 / 3, 1 / 3)
        x = synth.normal(60 + n, 1, T, K)
        blob = bn.pack("i2s", w.cuda())
        gap = 32 if n in (3, 4) else 0                     # a hole in the host block: no merging across it
        xh = xh_all[xo + gap: xo + gap + T * K].view(T, K)
        xh.copy_(x)
        yh = yh_all[yo: yo + T * M].view(T, M)
        xd = xd_all[xd_o: xd_o + T * K].view(T, K)
        yd = yd_all[yo: yo + T * M].view(T, M)
        xo += T * K + gap
        xd_o += T * K
        yo += T * M
        qd = torch.empty((T, K), dtype=torch.int8, device="cuda")
        sd = torch.empty(T, dtype=torch.float32, device="cuda")
        ws = bn.new_workspace("i2s", T, M, K)
        items.append(dict(fmt="i2s", packed=blob, w_scale=0.5, M=M, K=K, x_host=xh, y_host=yh, x_dev=xd, q_dev=qd,
                          scale_dev=sd, y_dev=yd, workspace=ws))
        keep.append((blob, qd, sd, ws))
        y, _, _, _ = bn.bitnet_linear("i2s", blob, 0.5, M, K, x.cuda())
        refs.append(y.cpu())
    assert xo <= nx + 64
    bn.bitnet_linear_host_batch(bn.make_host_batch(items))
    torch.cuda.current_stream().synchronize()
    for it, ref in zip(items, refs):
        assert torch.equal(it["y_host"], ref)
    assert bool((yh_all[ny:] == -7.0).all())
    assert bn.bitnet_device_status() == 0


@pytest.mark.parametrize("fmt", ["tl1", "tl2"])
def test_tl_workspace_shared_by_calls_of_different_shapes(fmt):
    """One workspace serves TL calls of different shapes back to back: the tables of a call with few rows lie
    where a later call with many rows keeps its split-K sums, so every call must clear what it relies on."""
    shapes = [(32, 28672, 2), (4096, 8192, 1), (64, 14336, 3), (2048, 28672, 1), (32, 96 * 40, 1)]
    bn.bitnet_set_tl2_lookup(True)     # the kernel that keeps tables and sums in the workspace, for both formats
    try:
        _shared_workspace_calls(fmt, shapes)
    finally:
        bn.bitnet_set_tl2_lookup(False)


def _shared_workspace_calls(fmt, shapes):
    n = max(bn.bitnet_mpgemm_workspace_bytes(fmt, T, M, K) for M, K, T in shapes)
    ws = torch.full((n,), 0x5A, dtype=torch.uint8, device="cuda")      # never initialised: garbage on purpose
    cases = []
    for i, (M, K, T) in enumerate(shapes):
        w = tern(90 + i, M, K)
        x = synth.normal(91, i, T, K)
        q, sc, _ = bn.bitnet_quant_act(x.cuda())
        cases.append((M, K, T, w, x, q, sc, bn.pack(fmt, w.cuda())))
    outs = []
    for M, K, T, w, x, q, sc, blob in cases + cases[::-1]:             # no synchronisation between the calls
        outs.append(bn.bitnet_mpgemm(fmt, blob, 0.5, M, K, q, sc, want_acc=True, workspace=ws))
    torch.cuda.synchronize()
    for (M, K, T, w, x, q, sc, blob), (y, acc) in zip(cases + cases[::-1], outs):
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(acc), acc_ref)
        check_y(y, acc_ref, sc_ref, 0.5)


def test_bounded_wait_times_out_and_reports():
    """A device-side wait that cannot complete gives up after its poll limit, sets the status flag and lets the kernel
    return: the context stays usable, bitnet_device_status reports the time-out, and the flag can be cleared."""
    assert bn.bitnet_device_status() == 0
    bn.bitnet_debug_wait_timeout_probe()
    assert bn.bitnet_device_status() == 6          # BITNET_ERR_TIMEOUT
    assert "wait" in bn.status_string(6)
    bn.bitnet_device_status_clear()
    assert bn.bitnet_device_status() == 0
    # the device still computes
    check_linear("tl1", tern(95, 32, 192), synth.normal(95, 1, 1, 192))


def _run_child(code, extra_env):
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    out = subprocess.run([sys.executable, "-c", code], cwd=root, env=dict(os.environ, **extra_env), capture_output=True,
                         text=True, timeout=900)
    assert out.returncode == 0 and "ok" in out.stdout, (extra_env, out.stderr[-2000:])


@pytest.mark.parametrize("extra", [dict(BITNET_PREFILL="simt"), dict(BITNET_PREFILL_TMA_STORE="0"),
                                   dict(BITNET_I2S_STREAM="ring"), dict(BITNET_QUANT_CLUSTERS="0"),
                                   dict(BITNET_FUSE_MAX_T="0"), dict(BITNET_I2S_MID_MIN_T="9"),
                                   dict(BITNET_MID_NS="5"), dict(BITNET_TL2="lut"), dict(BITNET_TL2_S="4", BITNET_TL2_DEPTH="4"),
                                   dict(BITNET_GROUP="0"), dict(BITNET_GROUP_S="2", BITNET_GROUP_DEPTH="8"),
                                   dict(BITNET_GROUP_DEPTH="12"), dict(BITNET_TL1="table")])
def test_read_once_switches_in_child_processes(extra):
    """Every kernel choice that an environment variable makes (read once per process) against the oracle: the dp4a
    prefill kernel, plain stores instead of bulk tensor stores in the tensor-core prefill kernel, the bulk-copy ring
    decode kernel, the quantiser without clusters, no fused quantiser, the mid-batch kernel's lower limit and forced
    slice count, the lookup-table kernel for TL1 and TL2, other ring depths and warps per unit in the grouped kernels,
    the grouped call switched off, and TL1 through the scan kernel's decode table instead of its arithmetic decode."""
    code = (
        "import sys; sys.path.insert(0, 'tests'); import numpy as np, torch\n"
        "import oracle\n"
        "from paper_2502_11880_b200 import synth\n"
        "import paper_2502_11880_b200 as bn\n"
        "from helpers import check_linear, check_y, run_fused, npy\n"
        "from test_gpu_group import Item, run_group\n"
        "for (M, K, T) in [(70, 1536, 1), (64, 8192, 2), (33, 28672, 5), (48, 16384, 6), (40, 8192, 8), (200, 4096, 20),\n"
        "                  (300, 2048, 300)]:\n"
        "    check_linear('i2s', synth.ternary(62, 1, M, K, 1/3, 1/3), synth.normal(62, T, T, K))\n"
        "for (M, K, T) in [(64, 3200, 1), (96, 8192, 3), (32, 28672, 8), (64, 130, 2)]:\n"
        "    for fmt in ('tl2', 'tl1'):\n"
        "        check_linear(fmt, synth.ternary(63, 1, M, K, 1/3, 1/3), synth.normal(63, T, T, K))\n"
        "for (M, K, T) in [(96, 8192, 1), (64, 28672, 4), (32, 16384, 7)]:\n"
        "    w = synth.ternary(64, 1, M, K, 1/3, 1/3); x = synth.normal(64, T, T, K)\n"
        "    for fmt in ('i2s', 'tl2'):\n"
        "        y, q, sc, acc = run_fused(fmt, bn.pack(fmt, w.cuda()), 0.5, M, K, x.cuda(), workspace=bn.new_workspace(fmt, T, M, K))\n"
        "        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())\n"
        "        assert np.array_equal(npy(q), q_ref) and np.array_equal(npy(acc), oracle.mpgemm_def(q_ref, w.numpy()))\n"
        "items = [Item('i2s', 160, 8192, 1, 900), Item('tl2', 64, 8192, 1, 901), Item('i2s', 48, 28672, 8, 902), Item('i2s', 2000, 2048, 3, 903),\n"
        "         Item('tl2', 640, 3200, 2, 904), Item('tl1', 96, 8192, 1, 905), Item('tl1', 320, 4096, 4, 906)]\n"
        "run_group(items)\n"
        "for it in items: it.check()\n"
        "assert bn.bitnet_device_status() == 0\n"
        "print('ok')\n")
    _run_child(code, extra)


@pytest.mark.parametrize("fmt", ["tl1", "tl2"])
def test_tl_prefill_through_the_transcode(fmt):
    """TL blobs at prefill batch sizes: the blob is turned into its I2_S form in the workspace (device-side transcode
    of the packed codes) and the tensor-core prefill kernel serves the call; accumulators equal the definition.  The
    transcoded bytes themselves must equal the I2_S packer's blob of the same matrix."""
    for i, (M, K, T) in enumerate([(320, 4096, 128), (64, 1536, 200), (160, 8640, 130), (96, 3200, 256), (32, 64, 128)]):
        w = tern(110 + i, M, K, 0.4, 0.3)
        x = synth.normal(111, i, T, K)
        q, sc, _ = bn.bitnet_quant_act(x.cuda())
        blob = bn.pack(fmt, w.cuda())
        ws = bn.new_workspace(fmt, T, M, K)
        assert ws.numel() >= bn.bitnet_i2s_packed_bytes(M, K)
        y, acc = bn.bitnet_mpgemm(fmt, blob, 0.5, M, K, q, sc, want_acc=True, workspace=ws)
        torch.cuda.synchronize()
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(acc), acc_ref), (fmt, M, K, T)
        check_y(y, acc_ref, sc_ref, 0.5)
        n = bn.bitnet_i2s_packed_bytes(M, K)
        assert np.array_equal(npy(ws[:n]), oracle.pack_i2s(w.numpy())), (fmt, M, K)
    assert bn.bitnet_device_status() == 0


@pytest.mark.parametrize("fmt", ["i2s", "tl1", "tl2"])
def test_pack_then_compute_back_to_back_on_one_stream(fmt):
    """A blob packed and used at once -- no host synchronisation between the packer and the first kernel that reads
    it, early start on: the decode and prefill kernels copy packed weights before they wait for earlier kernels, so
    the library itself must order the first launch after a packer behind it.  1, 16 and 256 tokens, through the
    quantiser (the launch that follows the packer is then not the one that reads the blob) and without it."""
    for i, (M, K, T) in enumerate([(4096, 8192, 1), (2048, 4096, 16), (1024, 4096, 256), (8192, 8192, 3)]):
        w = tern(130 + i, M, K)
        x = synth.normal(131, i, T, K)
        wd, xd = w.cuda(), x.cuda()
        q0, sc0, _ = bn.bitnet_quant_act(xd)
        ws = bn.new_workspace(fmt, T, M, K)
        ws2 = bn.new_workspace(fmt, T, M, K)
        torch.cuda.synchronize()
        blob = bn.pack(fmt, wd, check=False)
        y, acc = bn.bitnet_mpgemm(fmt, blob, 0.5, M, K, q0, sc0, want_acc=True, workspace=ws)
        blob2 = bn.pack(fmt, wd, check=False)
        y2, q2, sc2, acc2 = bn.bitnet_linear(fmt, blob2, 0.5, M, K, xd, want_acc=True, workspace=ws2)
        torch.cuda.synchronize()
        q_ref, sc_ref, _ = oracle.quant_act(x.numpy())
        acc_ref = oracle.mpgemm_def(q_ref, w.numpy())
        assert np.array_equal(npy(acc), acc_ref), (fmt, M, K, T)
        assert np.array_equal(npy(acc2), acc_ref), (fmt, M, K, T)
        check_y(y, acc_ref, sc_ref, 0.5)
        check_y(y2, acc_ref, sc_ref, 0.5)

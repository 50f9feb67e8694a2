"""Shared helpers of the GPU parity tests: run the CUDA path and the oracle on the same seeded inputs."""
import numpy as np
import torch

import oracle
import paper_2502_11880_b200 as bn

REL_TOL = 1e-6   # fp32 outputs against the oracle's float64 product (two fp32 roundings <= 2^-23)


def dev(a):
    return torch.as_tensor(a).cuda()


def npy(t):
    return t.detach().cpu().numpy()


def check_y(y_gpu, acc_ref, act_scale_ref, w_scale):
    """|y - y_ref| <= 1e-6 |y_ref| element-wise, and y == 0 exactly where the accumulator is 0."""
    y_ref = oracle.dequant(acc_ref, act_scale_ref, w_scale)
    y = npy(y_gpu).astype(np.float64)
    assert y.shape == y_ref.shape
    err = np.abs(y - y_ref)
    assert np.all(err <= REL_TOL * np.abs(y_ref)), float((err / np.maximum(np.abs(y_ref), 1e-300)).max())
    assert np.all(y[acc_ref == 0] == 0.0)


def oracle_pack(fmt, w_np, bk3=0):
    return oracle.pack_i2s(w_np) if fmt == "i2s" else oracle.pack_tl(fmt, w_np, bk3)


GUARD_BYTES = 256      # canary bytes on either side of every output buffer of run_linear (keeps 16-byte alignment)
CANARY = 0xA5


class Guarded:
    """An output tensor of the given shape and dtype inside a byte buffer with canaries on both sides:
    a kernel that writes a single byte outside its output is caught by `intact()`."""

    def __init__(self, shape, dtype):
        n = 1
        for d in shape:
            n *= int(d)
        self.nbytes = n * torch.empty((), dtype=dtype).element_size()
        self.buf = torch.full((self.nbytes + 2 * GUARD_BYTES,), CANARY, dtype=torch.uint8, device="cuda")
        self.t = self.buf[GUARD_BYTES: GUARD_BYTES + self.nbytes].view(dtype).view(*shape)

    def intact(self):
        lo, hi = self.buf[:GUARD_BYTES], self.buf[GUARD_BYTES + self.nbytes:]
        return bool((lo == CANARY).all()) and bool((hi == CANARY).all())


def run_linear(fmt, w_t, x_t, bk3=0, workspace=None, w_scale=None):
    """Full path on the GPU: quantise, pack, mpgemm, every output between canary bytes that are checked
    afterwards.  Returns dict of device tensors."""
    M, K = w_t.shape
    T = x_t.shape[0]
    wd, xd = w_t.cuda(), x_t.cuda()
    gq, gsc, gsm = Guarded((T, K), torch.int8), Guarded((T,), torch.float32), Guarded((T,), torch.int32)
    gy, gacc = Guarded((T, M), torch.float32), Guarded((T, M), torch.int32)
    q, sc, sm = bn.bitnet_quant_act(xd, q=gq.t, act_scale=gsc.t, act_sum=gsm.t)
    blob = bn.pack(fmt, wd, bk3)
    ws = bn.synth.absmean_scale(w_t) if w_scale is None else w_scale
    y, acc = bn.bitnet_mpgemm(fmt, blob, ws, M, K, q, sc, bk3=bk3, y=gy.t, acc_out=gacc.t, workspace=workspace)
    torch.cuda.synchronize()
    for name, g in (("q", gq), ("act_scale", gsc), ("act_sum", gsm), ("y", gy), ("acc", gacc)):
        assert g.intact(), f"{fmt} M={M} K={K} T={T}: bytes outside {name} were written"
    return dict(q=q, act_scale=sc, act_sum=sm, blob=blob, y=y, acc=acc, w_scale=ws)


def no_workspace():
    """An empty workspace: calls that would use one when offered (the I2_S mid-batch kernel for crowded decode
    batches) run the kernel that needs none instead."""
    return torch.empty(0, dtype=torch.uint8, device="cuda")


def run_fused(fmt, blob, w_scale, M, K, x_dev, workspace=None, bk3=0):
    """bitnet_linear (quantiser + mpGEMM from fp32 activations) with every output between canary bytes.
    Returns (y, q, act_scale, acc)."""
    T = x_dev.shape[0]
    gq, gsc = Guarded((T, K), torch.int8), Guarded((T,), torch.float32)
    gy, gacc = Guarded((T, M), torch.float32), Guarded((T, M), torch.int32)
    y, q, sc, acc = bn.bitnet_linear(fmt, blob, w_scale, M, K, x_dev, bk3=bk3, q=gq.t, act_scale=gsc.t, y=gy.t,
                                     acc_out=gacc.t, workspace=workspace)
    torch.cuda.synchronize()
    for name, g in (("q", gq), ("act_scale", gsc), ("y", gy), ("acc", gacc)):
        assert g.intact(), f"{fmt} M={M} K={K} T={T}: bitnet_linear wrote outside {name}"
    return y, q, sc, acc


def check_linear(fmt, w_t, x_t, bk3=0, rows=None, workspace=None):
    """Element-by-element parity of one linear layer against the oracle (all rows, or a sample)."""
    out = run_linear(fmt, w_t, x_t, bk3, workspace)
    w_np, x_np = w_t.numpy(), x_t.numpy()
    q_ref, sc_ref, sm_ref = oracle.quant_act(x_np)
    assert np.array_equal(npy(out["q"]), q_ref)
    assert np.array_equal(npy(out["act_scale"]).view(np.uint32), sc_ref.view(np.uint32))
    assert np.array_equal(npy(out["act_sum"]), sm_ref)
    assert np.array_equal(npy(out["blob"]), oracle_pack(fmt, w_np, bk3))
    acc_ref = oracle.mpgemm_def(q_ref, w_np)
    assert np.array_equal(npy(out["acc"]), acc_ref)
    check_y(out["y"], acc_ref, sc_ref, out["w_scale"])
    return out

"""Runs one linear layer of a given shape a few times on cuda:0 (an example of the Python binding, and the
small, self-contained workload the ncu captures under profiles/ are taken on).

    python -m paper_2502_11880_b200.run_case FMT K M T [N] [--two-kernel]

FMT = i2s | tl1 | tl2.  Weights and activations are seeded synthetic tensors; N launches (default 6) over
three distinct copies of the packed blob.  T <= 8 runs the decode path through bitnet_linear (one fused kernel
for I2_S up to 5 tokens unless --two-kernel); larger T runs the quantiser and bitnet_mpgemm: the mid-batch
kernel up to 64 tokens (large tensors from 33 tokens on: the streaming tcgen05 kernel, unless
BITNET_I2S_STREAM_TC=0), the prefill kernel beyond.
"""
import sys

import torch

import paper_2502_11880_b200 as bn
from paper_2502_11880_b200 import synth


def main(argv):
    two = "--two-kernel" in argv
    argv = [a for a in argv if not a.startswith("--")]
    fmt, K, M, T = argv[0], int(argv[1]), int(argv[2]), int(argv[3])
    n = int(argv[4]) if len(argv) > 4 else 6
    w = synth.ternary(7, 1, M, K, 1 / 3, 1 / 3, device="cuda")
    blobs = [bn.pack(fmt, w, check=False) for _ in range(3)]
    w_scale = synth.absmean_scale(w)
    del w
    x = synth.normal(7, 2, T, K).cuda()
    q, sc, sm = bn.bitnet_quant_act(x)
    y = torch.empty((T, M), dtype=torch.float32, device="cuda")
    ws = bn.new_workspace(fmt, T, M, K)
    torch.cuda.synchronize()
    for i in range(n):
        if two or T > 8:
            bn.bitnet_quant_act(x, q=q, act_scale=sc, act_sum=sm)
            bn.bitnet_mpgemm(fmt, blobs[i % 3], w_scale, M, K, q, sc, y=y, workspace=ws)
        else:
            bn.bitnet_linear(fmt, blobs[i % 3], w_scale, M, K, x, q=q, act_scale=sc, y=y, workspace=ws)
    torch.cuda.synchronize()
    print("done; device status", bn.bitnet_device_status(), "; y[0,:4] =", y[0, :4].tolist())


if __name__ == "__main__":
    main(sys.argv[1:])

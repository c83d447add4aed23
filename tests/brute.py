"""Independent brute-force restatements used to pin the oracle (numpy, tiny sizes only).

`unfold_matmul_conv` follows Eq. 5 of the paper: build the unfolded input U(X) with
explicit zero padding and multiply by the weight matrix.  It shares nothing with the
oracle's C loops: different language, different formulation (materialised unfold +
matrix product instead of a direct nested sum).
"""
import numpy as np


def bf16_to_f64(bits):
    b = np.asarray(bits, dtype=np.uint16).astype(np.uint32) << 16
    return b.view(np.float32).astype(np.float64)


def f32_to_bf16_bits(a):
    """Round-to-nearest-even fp32 -> bf16 bit patterns (finite inputs)."""
    u = np.asarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    r = u + 0x7FFF + ((u >> 16) & 1)
    return (r >> 16).astype(np.uint16)


def unfold_matmul_conv(x, w, stride=(1, 1), pad=(0, 0), dil=(1, 1)):
    """x [N,H,W,C] fp64, w [Co,KH,KW,C] fp64 -> y [N,Ho,Wo,Co] fp64 via Y = W U(X)."""
    N, H, W, C = x.shape
    Co, KH, KW, _ = w.shape
    xp = np.zeros((N, H + 2 * pad[0], W + 2 * pad[1], C))
    xp[:, pad[0]:pad[0] + H, pad[1]:pad[1] + W, :] = x
    Ho = (H + 2 * pad[0] - dil[0] * (KH - 1) - 1) // stride[0] + 1
    Wo = (W + 2 * pad[1] - dil[1] * (KW - 1) - 1) // stride[1] + 1
    cols = np.zeros((KH * KW * C, N * Ho * Wo))
    col = 0
    for n in range(N):
        for i in range(Ho):
            for j in range(Wo):
                patch = np.empty((KH, KW, C))
                for u in range(KH):
                    for s in range(KW):
                        patch[u, s, :] = xp[n, i * stride[0] + u * dil[0], j * stride[1] + s * dil[1], :]
                cols[:, col] = patch.reshape(-1)
                col += 1
    Y = w.reshape(Co, -1) @ cols
    return Y.T.reshape(N, Ho, Wo, Co)

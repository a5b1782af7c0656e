"""Test-side reference for the BF16 tensor-core gradient path: Eq. 2 in double precision on operands
rounded to bfloat16 at exactly the points where the CUDA path rounds them.

This is neither the oracle (which stays in double on the fp32 master values) nor product code: it exists
so that the tensor-core kernels can be pinned element-wise far below bf16 rounding.  What is left between
it and the GPU is fp32 accumulation order (about 1e-6 relative) and the rare activation or dZ entry whose
fp32 value sits on a bf16 rounding boundary.

Rounding points of the CUDA path (stated precision of the library):
  A_0            = bf16(features of the mini-batch)
  W_l^h          = bf16(W_l) for every layer but the last; biases and the last layer stay fp32
  A_{l+1}        = bf16(ReLU(A_l W_l^h^T + b_l))                      (fp32 accumulate, fp32 bias)
  logits         = A_{L-1} W_{L-1}^T + b_{L-1}                        (fp32 master weights)
  dZ_L           = (softmax - onehot) / B                             (fp32)
  dW_{L-1}, db   = dZ_L^T A_{L-1}, column sums of dZ_L                (fp32)
  dZ_{L-1}       = bf16((dZ_L W_{L-1}) * [A_{L-1} > 0])
  dW_l, db_l     = dZ_{l+1}^T A_l, column sums of dZ_{l+1}            (bf16 operands, fp32 accumulate)
  dZ_l           = bf16((dZ_{l+1} W_l^h) * [A_l > 0])
"""
from __future__ import annotations

import numpy as np


def bf16_round(a) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even), returned as float64."""
    a32 = np.ascontiguousarray(a, dtype=np.float32)
    u = a32.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).astype(np.float64).reshape(a32.shape)


def mlp_grad_bf16_points(x, layers, feats, labels):
    """(g, loss) in the layout of x, with the rounding points listed in the module docstring."""
    x = np.asarray(x, dtype=np.float32)            # fp32 master parameters
    L = len(layers) - 1
    Ws, bs = [], []
    off = 0
    for l in range(L):
        fin, fout = layers[l], layers[l + 1]
        Ws.append(x[off: off + fout * fin].astype(np.float64).reshape(fout, fin))
        off += fout * fin
        bs.append(x[off: off + fout].astype(np.float64))
        off += fout
    labels = np.asarray(labels)
    B = len(labels)
    A = [bf16_round(feats)]
    Wh = [bf16_round(Ws[l]) for l in range(L - 1)]
    for l in range(L - 1):
        A.append(bf16_round(np.maximum(A[l] @ Wh[l].T + bs[l], 0.0)))
    logits = A[L - 1] @ Ws[L - 1].T + bs[L - 1]
    zmax = logits.max(axis=1, keepdims=True)
    e = np.exp(logits - zmax)
    lse = zmax[:, 0] + np.log(e.sum(axis=1))
    loss = float(np.mean(lse - logits[np.arange(B), labels]))
    dz = e / e.sum(axis=1, keepdims=True)
    dz[np.arange(B), labels] -= 1.0
    dz /= B
    grads = [None] * L
    grads[L - 1] = (dz.T @ A[L - 1], dz.sum(axis=0))
    if L >= 2:
        dz = bf16_round((dz @ Ws[L - 1]) * (A[L - 1] > 0.0))
    for l in range(L - 2, -1, -1):
        grads[l] = (dz.T @ A[l], dz.sum(axis=0))
        if l >= 1:
            dz = bf16_round((dz @ Wh[l]) * (A[l] > 0.0))
    g = np.concatenate([np.concatenate([gw.ravel(), gb]) for gw, gb in grads])
    return g, loss

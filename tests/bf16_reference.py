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


def mlp_grad_bf16_points(x, layers, feats, labels, flips=(), ambiguous=None, details=None):
    """(g, loss) in the layout of x, with the rounding points listed in the module docstring.

    The ReLU decision A > 0 is taken on a sum the CUDA path accumulates in fp32 and this function in double:
    where a pre-activation is closer to zero than fp32 accumulation can resolve, both decisions are legitimate.
    `ambiguous`, if a list, receives those entries as (layer, sample, unit) (layer = index of the activation,
    1 .. L-1); `flips` names entries whose decision is inverted; `details`, if a dict, receives the activations
    "A" (list) and the back-propagated dA before the ReLU mask, "dA" (dict by layer)."""
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
        z = A[l] @ Wh[l].T + bs[l]
        if ambiguous is not None:
            # What the CUDA path's pre-activation may differ by: fp32 accumulation of K exact products on the tensor
            # cores, and, from the second layer on, input activations that rounded to the neighbouring bf16 value
            # (one unit in the last place, 2^-8, of a term).  1e-4 of the sum of the terms' magnitudes covers both;
            # the set only says where a decision MAY differ, the CUDA path's output says whether it does.
            resolve = 1e-4 * (np.abs(A[l]) @ np.abs(Wh[l]).T + np.abs(bs[l]))
            for s_, u_ in zip(*np.nonzero(np.abs(z) <= resolve)):
                ambiguous.append((l + 1, int(s_), int(u_)))
        a_next = bf16_round(np.maximum(z, 0.0))
        for (fl, s_, u_) in flips:
            if fl == l + 1:
                a_next[s_, u_] = 0.0 if a_next[s_, u_] > 0.0 else 2.0 ** -100    # off, or on with a negligible value
        A.append(a_next)
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
    pre_mask = {}
    if L >= 2:
        pre_mask[L - 1] = dz @ Ws[L - 1]
        dz = bf16_round(pre_mask[L - 1] * (A[L - 1] > 0.0))
    for l in range(L - 2, -1, -1):
        grads[l] = (dz.T @ A[l], dz.sum(axis=0))
        if l >= 1:
            pre_mask[l] = dz @ Wh[l]
            dz = bf16_round(pre_mask[l] * (A[l] > 0.0))
    if details is not None:
        details["A"], details["dA"] = A, pre_mask
    g = np.concatenate([np.concatenate([gw.ravel(), gb]) for gw, gb in grads])
    return g, loss


def block_errors(layers, got, ref, tol):
    """Per layer block (W_l, b_l), worst over the blocks: (max element-wise error / block max-norm,
    2-norm error / block 2-norm, fraction of the block's entries whose error exceeds tol x block max-norm)."""
    mx, l2, frac, off = 0.0, 0.0, 0.0, 0
    for l in range(len(layers) - 1):
        for size in (layers[l] * layers[l + 1], layers[l + 1]):
            a, r = got[off:off + size], ref[off:off + size]
            scale = max(np.abs(r).max(), 1e-30)
            e = np.abs(a - r)
            mx = max(mx, float(e.max() / scale))
            l2 = max(l2, float(np.linalg.norm(a - r) / max(np.linalg.norm(r), 1e-30)))
            frac = max(frac, float(np.count_nonzero(e > tol * scale)) / size)
            off += size
    return mx, l2, frac


def block_error(layers, got, ref):
    return block_errors(layers, got, ref, 0.0)[0]


def gradient_agrees(got, x, layers, feats, labels, tol=5e-3, tol_l2=1e-3):
    """Does a gradient row computed by the CUDA path agree with the reference?  Returns (ok, report).

    The gate, per layer block (W_l, b_l): every entry within tol of the block's max-norm and the block's 2-norm
    error within tol_l2 of its 2-norm.  (An activation or dZ entry that lands on the other side of a bf16 rounding
    boundary, which fp32 versus double accumulation decides, moves one row of a weight gradient by about 2^-8 of
    one sample's share: up to about 1e-3 of the block's max-norm per such entry (measured worst over the test
    shapes and the full-size runs: 3.2e-3 on a single row), next to nothing in the 2-norm (measured <= 4.5e-4).  A
    dropped K block, a mis-scaled bias gradient or wrong masks on a few percent of the entries are orders of
    magnitude above both bars.)  When the gate fails and the reference
    reports ReLU decisions that fp32 accumulation cannot resolve, each of them is a legitimate result either way,
    and the decision the CUDA path took can be read off its output: switching the decision of (layer l, sample s,
    unit u) changes row u of dW_{l-1} by dA_l[s, u] * A_{l-1}[s, :].  The residual of every such row is fitted
    (least squares over the row's ambiguous samples) with those terms; a fitted coefficient nearer to the
    switch than to zero switches the decision.  The reference is then recomputed with the inferred decisions and
    the same gate applied.  Decisions outside the ambiguous set are never touched."""
    amb, det = [], {}
    g, loss = mlp_grad_bf16_points(x, layers, feats, labels, ambiguous=amb, details=det)
    mx, l2, frac = block_errors(layers, got, g, tol)
    report = dict(max=mx, l2=l2, frac=frac, ambiguous=len(amb), switched=0, loss=loss)
    if mx <= tol and l2 <= tol_l2:
        return True, report
    if not amb:
        return False, report
    w_off, off = [], 0
    for l in range(len(layers) - 1):
        w_off.append(off)
        off += layers[l] * layers[l + 1] + layers[l + 1]
    rows = {}
    for (l, s_, u_) in amb:
        rows.setdefault((l, u_), []).append(s_)
    flips = []
    for (l, u_), samples in rows.items():
        fin = layers[l - 1]
        lo = w_off[l - 1] + u_ * fin
        resid = got[lo: lo + fin] - g[lo: lo + fin]
        basis = np.stack([det["A"][l - 1][s_] for s_ in samples], axis=1)          # fin x candidates
        coef, *_ = np.linalg.lstsq(basis, resid, rcond=None)
        for s_, c in zip(samples, coef):
            term = bf16_round(det["dA"][l][s_, u_])
            switch = -term if det["A"][l][s_, u_] > 0.0 else term      # what switching this decision adds to the row
            if switch != 0.0 and abs(c - switch) < abs(c):
                flips.append((l, s_, u_))
    report["switched"] = len(flips)
    if not flips:
        return False, report
    g2, loss2 = mlp_grad_bf16_points(x, layers, feats, labels, flips=flips)
    mx2, l22, frac2 = block_errors(layers, got, g2, tol)
    report.update(max=mx2, l2=l22, frac=frac2, loss=loss2)
    return (mx2 <= tol and l22 <= tol_l2), report

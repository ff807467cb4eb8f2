"""CPU oracle for Bi-Level Routing Attention (BRA).  TEST INFRASTRUCTURE ONLY.

A plain, slow, fp64 NumPy statement of what the hot path computes, written
from the paper (BiFormer, arXiv 2303.08810) step by step in its own order and
notation.  It shares no code with the CUDA path and never imports it; only
tests, the smoke check and the benchmark's CPU-baseline leg may import it.

Every function is pinned by the CPU tests (brute force on tiny inputs,
closed forms, special cases that reduce to textbook full attention, a library
correlation routine, finite differences).  Nothing in this file is
"parity unpinned".

Conventions (the paper is silent on these; the readings are listed in the
design notes of the repository):
  * tensors are [B, H, W, C]; channel c = head * d + j (Eq. 2 concat order)
  * regions are numbered row-major, r = ry * S + rx; tokens inside a region
    are in raster order (the reshape of "region partition", Section 3.2)
  * routing is per head (affinity summed over that head's d channels) unless
    shared_routing is set, in which case Eq. 4 is read literally over all C
  * top-k order: score descending, ties to the lower region index
  * LCE: 5x5 depthwise cross-correlation over the whole H x W map of V,
    stride 1, zero padding 2 (Section 3.2, Eq. 7)
  * a map whose sides S does not divide (Appendix C only says that S is chosen
    as a divisor "to avoid padding"): Q, K, V are zero-padded at the bottom and
    right to the next multiples of S, the padded map is processed as any other
    (the zero tokens are pooled, routed to and attended to like real ones),
    and O, lse and the gradients are cropped back
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------
# Region partition ("patchify" / "unpatchify", Algorithm 1 first and last step)
# ----------------------------------------------------------------------------
def region_partition(X, S):
    """[B,H,W,C] -> [B, S^2, HW/S^2, C] (Section 3.2, region partition)."""
    B, H, W, C = X.shape
    if H % S or W % S:
        raise ValueError("S must divide H and W")
    hs, ws = H // S, W // S
    Xr = X.reshape(B, S, hs, S, ws, C)          # (b, ry, y, rx, x, c)
    Xr = Xr.transpose(0, 1, 3, 2, 4, 5)         # (b, ry, rx, y, x, c)
    return Xr.reshape(B, S * S, hs * ws, C)


def region_unpartition(Xr, S, H, W):
    """Inverse of region_partition: [B, S^2, n_r, C] -> [B,H,W,C]."""
    B, R, n_r, C = Xr.shape
    hs, ws = H // S, W // S
    X = Xr.reshape(B, S, S, hs, ws, C).transpose(0, 1, 3, 2, 4, 5)
    return X.reshape(B, H, W, C)


# ----------------------------------------------------------------------------
# Region-to-region routing (Section 3.2; Eq. 4, Eq. 5)
# ----------------------------------------------------------------------------
def region_means(X, S):
    """Per-region average, Q^r / K^r in R^{S^2 x C}: [B,H,W,C] -> [B,S^2,C]."""
    Xr = region_partition(np.asarray(X, dtype=F64), S)
    n_r = Xr.shape[2]
    return Xr.sum(axis=2) / n_r


def region_affinity(Qr, Kr, heads, shared_routing=False):
    """Eq. 4, A^r = Q^r (K^r)^T, per head: [B,S^2,C] x2 -> [B,heads|1,S^2,S^2]."""
    B, R, C = Qr.shape
    if shared_routing:
        A = np.empty((B, 1, R, R), dtype=F64)
        for b in range(B):
            A[b, 0] = Qr[b] @ Kr[b].T
        return A
    d = C // heads
    A = np.empty((B, heads, R, R), dtype=F64)
    for b in range(B):
        for h in range(heads):
            A[b, h] = Qr[b, :, h * d:(h + 1) * d] @ Kr[b, :, h * d:(h + 1) * d].T
    return A


def topk_index(A, k):
    """Eq. 5, row-wise topkIndex: [..., R, R] -> int32 [..., R, k].

    Order inside a row: score descending, equal scores by ascending region
    index.  Also returns gap_rel [..., R]: the relative gap between the k-th
    and (k+1)-th score of each row (inf when k == R), used by the parity
    tests to find rows whose selection an fp32 evaluation may flip.
    """
    R = A.shape[-1]
    if not 1 <= k <= R:
        raise ValueError("topk must be in [1, S^2]")
    flat = A.reshape(-1, R)
    idx = np.empty((flat.shape[0], k), dtype=np.int32)
    gap = np.full((flat.shape[0],), np.inf, dtype=F64)
    cols = np.arange(R)
    for i in range(flat.shape[0]):
        row = flat[i]
        order = np.lexsort((cols, -row))        # primary: -score, secondary: index
        idx[i] = order[:k]
        if k < R:
            a, b = row[order[k - 1]], row[order[k]]
            gap[i] = (a - b) / max(abs(a), abs(b), 1e-30)
    return idx.reshape(A.shape[:-1] + (k,)), gap.reshape(A.shape[:-1])


# ----------------------------------------------------------------------------
# Token-to-token attention over the routed regions (Eq. 6, Eq. 7 with Eq. 1)
# ----------------------------------------------------------------------------
def routed_attention(Q, K, V, index, heads, S, scale):
    """Attention(Q, K^g, V^g) per query region and head.

    index: int [B, heads|1, S^2, k].  Row i lists the key regions whose
    tokens query region i attends to; it is a list (duplicates count twice,
    any order).  Returns (O_att [B,H,W,C], lse [B,heads,H*W]) where lse is
    the log of the softmax denominator of each (query, head), in the token's
    position y*W+x.
    """
    Q = np.asarray(Q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    B, H, W, C = Q.shape
    d = C // heads
    R = S * S
    Qp, Kp, Vp = region_partition(Q, S), region_partition(K, S), region_partition(V, S)
    n_r = Qp.shape[2]
    Op = np.empty_like(Qp)
    lse_p = np.empty((B, heads, R, n_r), dtype=F64)
    for b in range(B):
        for h in range(heads):
            ch = slice(h * d, (h + 1) * d)
            hi = 0 if index.shape[1] == 1 else h
            for i in range(R):
                regions = index[b, hi, i]
                if regions.min() < 0 or regions.max() >= R:
                    raise IndexError("routing index out of range")
                Kg = Kp[b, regions][:, :, ch].reshape(-1, d)      # Eq. 6 gather
                Vg = Vp[b, regions][:, :, ch].reshape(-1, d)
                s = scale * (Qp[b, i, :, ch] @ Kg.T)              # [n_r, k*n_r]
                m = s.max(axis=1, keepdims=True)
                e = np.exp(s - m)
                z = e.sum(axis=1, keepdims=True)
                Op[b, i, :, ch] = (e / z) @ Vg                    # Eq. 1 softmax(.) V
                lse_p[b, h, i] = (m + np.log(z))[:, 0]
    O = region_unpartition(Op, S, H, W)
    lse = region_unpartition(lse_p.transpose(0, 2, 3, 1), S, H, W)   # [B,H,W,heads]
    lse = lse.transpose(0, 3, 1, 2).reshape(B, heads, H * W)
    return O, lse


def lce(V, w, bias=None):
    """LCE(V): depthwise 5x5 cross-correlation, zero padding 2 (Eq. 7).

    out[b,y,x,c] = sum_{i,j<5} w[c,i,j] * V[b, y+i-2, x+j-2, c]  (+ bias[c]).
    """
    V = np.asarray(V, dtype=F64)
    w = np.asarray(w, dtype=F64)
    B, H, W, C = V.shape
    ks = w.shape[1]
    p = ks // 2
    Vp = np.zeros((B, H + 2 * p, W + 2 * p, C), dtype=F64)
    Vp[:, p:p + H, p:p + W] = V
    out = np.zeros((B, H, W, C), dtype=F64)
    for i in range(ks):
        for j in range(ks):
            out += w[:, i, j] * Vp[:, i:i + H, j:j + W, :]
    if bias is not None:
        out += np.asarray(bias, dtype=F64)
    return out


# ----------------------------------------------------------------------------
# Maps that S does not divide (Appendix C): zero padding, then cropping
# ----------------------------------------------------------------------------
def padded_size(H, W, S):
    """Next multiples of S."""
    return -(-H // S) * S, -(-W // S) * S


def pad_map(X, S):
    """[B,H,W,C] -> [B,Hp,Wp,C]: zeros appended at the bottom and at the right."""
    X = np.asarray(X, dtype=F64)
    B, H, W, C = X.shape
    Hp, Wp = padded_size(H, W, S)
    out = np.zeros((B, Hp, Wp, C), dtype=F64)
    out[:, :H, :W] = X
    return out


def crop_map(X, H, W):
    """The top-left H x W tokens of a padded map."""
    return np.ascontiguousarray(X[:, :H, :W])


def _crop_lse(lse, Hp, Wp, H, W):
    B, heads, _ = lse.shape
    return np.ascontiguousarray(lse.reshape(B, heads, Hp, Wp)[:, :, :H, :W]).reshape(B, heads, H * W)


# ----------------------------------------------------------------------------
# The four calls of the boundary, on host arrays
# ----------------------------------------------------------------------------
def default_scale(C, heads):
    return 1.0 / np.sqrt(C // heads)


def bra_route(Q, K, heads, S, topk, shared_routing=False):
    """Q, K -> (Q^r, K^r [B,S^2,C], I^r int32 [B,heads|1,S^2,k], gap_rel)."""
    if Q.shape[1] % S or Q.shape[2] % S:
        Q, K = pad_map(Q, S), pad_map(K, S)
    Qr, Kr = region_means(Q, S), region_means(K, S)
    A = region_affinity(Qr, Kr, heads, shared_routing)
    index, gap = topk_index(A, topk)
    return Qr, Kr, index, gap


def bra_attend(Q, K, V, index, w, heads, S, scale=None, bias=None):
    """Eq. 7: O = Attention(Q, K^g, V^g) + LCE(V).  w=None disables LCE."""
    H, W = Q.shape[1], Q.shape[2]
    if H % S or W % S:
        Hp, Wp = padded_size(H, W, S)
        O, lse = bra_attend(pad_map(Q, S), pad_map(K, S), pad_map(V, S), index, w, heads, S, scale, bias)
        return crop_map(O, H, W), _crop_lse(lse, Hp, Wp, H, W)
    C = Q.shape[-1]
    scale = default_scale(C, heads) if scale is None else scale
    O, lse = routed_attention(Q, K, V, index, heads, S, scale)
    if w is not None:
        O = O + lce(V, w, bias)
    return O, lse


def bra_forward(Q, K, V, w, heads, S, topk, scale=None, shared_routing=False, bias=None):
    """Algorithm 1 from the projected Q, K, V on: route, gather, attend, LCE."""
    _, _, index, gap = bra_route(Q, K, heads, S, topk, shared_routing)
    O, lse = bra_attend(Q, K, V, index, w, heads, S, scale, bias)
    return O, index, lse, gap


def bra_backward(Q, K, V, index, w, dO, heads, S, scale=None):
    """Gradients of sum(O * dO) for a fixed routing index.

    The index is a constant (top-k is not differentiable), so nothing flows
    through pooling or the affinity.  With P the softmax of Eq. 1 over the
    gathered keys: dV^g = P^T dO, dP = dO V^g^T, dS = P o (dP - rowsum(P o dP)),
    dQ = scale dS K^g, dK^g = scale dS^T Q; dK^g, dV^g rows are added back to
    the tokens of the regions they were gathered from.  LCE is linear in V and
    w: dV += correlation-transpose(dO, w), dw[c,i,j] = sum dO[.,y,x,c] V[.,y+i-2,x+j-2,c].
    Returns dQ, dK, dV [B,H,W,C], dw [C,5,5], dbias [C].
    """
    if np.shape(Q)[1] % S or np.shape(Q)[2] % S:
        H0, W0 = np.shape(Q)[1], np.shape(Q)[2]
        g = bra_backward(pad_map(Q, S), pad_map(K, S), pad_map(V, S), index, w, pad_map(dO, S), heads, S, scale)
        return crop_map(g[0], H0, W0), crop_map(g[1], H0, W0), crop_map(g[2], H0, W0), g[3], g[4]
    Q = np.asarray(Q, dtype=F64)
    K = np.asarray(K, dtype=F64)
    V = np.asarray(V, dtype=F64)
    dO = np.asarray(dO, dtype=F64)
    B, H, W, C = Q.shape
    d = C // heads
    R = S * S
    scale = default_scale(C, heads) if scale is None else scale
    Qp, Kp, Vp = region_partition(Q, S), region_partition(K, S), region_partition(V, S)
    dOp = region_partition(dO, S)
    n_r = Qp.shape[2]
    dQp, dKp, dVp = np.zeros_like(Qp), np.zeros_like(Kp), np.zeros_like(Vp)
    k = index.shape[-1]
    for b in range(B):
        for h in range(heads):
            ch = slice(h * d, (h + 1) * d)
            hi = 0 if index.shape[1] == 1 else h
            for i in range(R):
                regions = index[b, hi, i]
                Kg = Kp[b, regions][:, :, ch].reshape(-1, d)
                Vg = Vp[b, regions][:, :, ch].reshape(-1, d)
                q = Qp[b, i, :, ch]
                do = dOp[b, i, :, ch]
                s = scale * (q @ Kg.T)
                s -= s.max(axis=1, keepdims=True)
                P = np.exp(s)
                P /= P.sum(axis=1, keepdims=True)
                dVg = P.T @ do
                dP = do @ Vg.T
                dS = P * (dP - (P * dP).sum(axis=1, keepdims=True))
                dQp[b, i, :, ch] = scale * (dS @ Kg)
                dKg = scale * (dS.T @ q)
                for m in range(k):                      # scatter back, duplicates add
                    r = regions[m]
                    dKp[b, r, :, ch] += dKg[m * n_r:(m + 1) * n_r]
                    dVp[b, r, :, ch] += dVg[m * n_r:(m + 1) * n_r]
    dQ = region_unpartition(dQp, S, H, W)
    dK = region_unpartition(dKp, S, H, W)
    dV = region_unpartition(dVp, S, H, W)
    dw = np.zeros((C, 5, 5), dtype=F64)
    dbias = dO.sum(axis=(0, 1, 2))
    if w is not None:
        w = np.asarray(w, dtype=F64)
        p = 2
        Vpad = np.zeros((B, H + 2 * p, W + 2 * p, C), dtype=F64)
        Vpad[:, p:p + H, p:p + W] = V
        dOpad = np.zeros_like(Vpad)
        dOpad[:, p:p + H, p:p + W] = dO
        for i in range(5):
            for j in range(5):
                dw[:, i, j] = (dO * Vpad[:, i:i + H, j:j + W]).sum(axis=(0, 1, 2))
                # V[y', x'] receives w[i,j] * dO[y'-i+2, x'-j+2]
                dV += w[:, i, j] * dOpad[:, 4 - i:4 - i + H, 4 - j:4 - j + W]
    return dQ, dK, dV, dw, dbias


def keys_per_query(H, W, S, topk):
    """Number of key/value pairs each query attends to: k * HW / S^2."""
    return topk * (H // S) * (W // S)

"""Pins for the CPU oracle: what the paper and the mathematics fix.

None of these tests re-types the oracle's formulas with the same library
calls: each compares against brute-force Python loops over tokens, a closed
form, a special case that reduces to textbook full attention, a library
routine (scipy correlate2d, torch autograd / conv2d), finite differences, or a
value the paper prints (tests/golden).
"""
import itertools
import math
import os

import numpy as np
import pytest

from oracle import bra_oracle as orc

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.Generator(np.random.PCG64(seed))


def region_of(y, x, H, W, S):
    return (y // (H // S)) * S + (x // (W // S))


# ---------------------------------------------------------------- partition
def test_partition_places_every_token_by_hand():
    B, H, W, C, S = 2, 6, 4, 3, 2
    X = rng(1).standard_normal((B, H, W, C))
    Xr = orc.region_partition(X, S)
    hs, ws = H // S, W // S
    assert Xr.shape == (B, S * S, hs * ws, C)
    for b, y, x in itertools.product(range(B), range(H), range(W)):
        r = region_of(y, x, H, W, S)
        t = (y % hs) * ws + (x % ws)
        assert np.array_equal(Xr[b, r, t], X[b, y, x])
    assert np.array_equal(orc.region_unpartition(Xr, S, H, W), X)


def test_partition_rejects_non_divisor():
    with pytest.raises(ValueError):
        orc.region_partition(np.zeros((1, 7, 8, 2)), 2)


# ---------------------------------------------------------------- Eq. 10 / Eq. 4
def test_affinity_is_mean_of_all_token_pair_products():
    """Appendix A identity: mean over token pairs of Q_i.K_j == Q^r . K^r."""
    B, H, W, C, S, heads = 1, 4, 6, 4, 2, 2
    g = rng(2)
    Q, K = g.standard_normal((B, H, W, C)), g.standard_normal((B, H, W, C))
    Qr, Kr = orc.region_means(Q, S), orc.region_means(K, S)
    A = orc.region_affinity(Qr, Kr, heads)
    A_shared = orc.region_affinity(Qr, Kr, heads, shared_routing=True)
    d = C // heads
    toks = [(y, x) for y in range(H) for x in range(W)]
    R = S * S
    brute = np.zeros((heads, R, R))
    count = np.zeros((R, R))
    for (y1, x1) in toks:
        for (y2, x2) in toks:
            i, j = region_of(y1, x1, H, W, S), region_of(y2, x2, H, W, S)
            count[i, j] += 1
            for h in range(heads):
                acc = 0.0
                for c in range(h * d, (h + 1) * d):
                    acc += Q[0, y1, x1, c] * K[0, y2, x2, c]
                brute[h, i, j] += acc
    brute /= count
    np.testing.assert_allclose(A[0], brute, rtol=1e-12, atol=1e-12)
    np.testing.assert_allclose(A_shared[0, 0], brute.sum(axis=0), rtol=1e-12, atol=1e-12)
    # a transposed operand (K^r Q^r^T) would fail: the matrix is not symmetric
    assert not np.allclose(brute[0], brute[0].T)


# ---------------------------------------------------------------- Eq. 5
def test_topk_matches_python_sort_and_special_cases():
    g = rng(3)
    A = g.standard_normal((2, 3, 9, 9))
    for k in (1, 4, 9):
        idx, gap = orc.topk_index(A, k)
        assert idx.dtype == np.int32 and idx.shape == (2, 3, 9, k)
        for b, h, i in itertools.product(range(2), range(3), range(9)):
            row = A[b, h, i]
            expect = sorted(range(9), key=lambda j: (-row[j], j))[:k]
            assert list(idx[b, h, i]) == expect
            if k == 1:
                assert idx[b, h, i, 0] == int(np.argmax(row))
            if k == 9:
                assert sorted(idx[b, h, i]) == list(range(9))
                assert gap[b, h, i] == np.inf
            else:
                srt = sorted(row, reverse=True)
                assert gap[b, h, i] == pytest.approx(
                    (srt[k - 1] - srt[k]) / max(abs(srt[k - 1]), abs(srt[k])))


def test_topk_tie_break_lower_index_first():
    A = np.array([[[1.0, 3.0, 3.0, 0.0],
                   [2.0, 2.0, 2.0, 2.0],
                   [0.0, -1.0, 5.0, 5.0],
                   [-0.0, 0.0, -1.0, -2.0]]])
    idx, gap = orc.topk_index(A, 2)
    assert idx.tolist() == [[[1, 2], [0, 1], [2, 3], [0, 1]]]
    assert gap[0, 1] == 0.0
    idx3, _ = orc.topk_index(A, 3)
    assert idx3[0, 0].tolist() == [1, 2, 0]


def test_topk_rejects_bad_k():
    with pytest.raises(ValueError):
        orc.topk_index(np.zeros((4, 4)), 0)
    with pytest.raises(ValueError):
        orc.topk_index(np.zeros((4, 4)), 5)


# ---------------------------------------------------------------- Table 7
def test_keys_per_query_reproduces_the_papers_table():
    rows = 0
    with open(os.path.join(GOLDEN, "table7_tokens_to_attend.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            maps, Ss, ks, toks = ([int(v) for v in part.split(",")] for part in line.split("|"))
            for m, S, k, t in zip(maps, Ss, ks, toks):
                assert orc.keys_per_query(m, m, S, k) == t
            rows += 1
    assert rows == 5


# ---------------------------------------------------------------- attention
def full_attention_loops(Q, K, V, heads, scale):
    """Textbook softmax attention over all tokens, one query at a time."""
    B, H, W, C = Q.shape
    d = C // heads
    O = np.zeros_like(Q)
    lse = np.zeros((B, heads, H * W))
    Kf, Vf = K.reshape(B, H * W, C), V.reshape(B, H * W, C)
    for b in range(B):
        for h in range(heads):
            for y in range(H):
                for x in range(W):
                    q = Q[b, y, x, h * d:(h + 1) * d]
                    s = np.array([scale * float(np.dot(q, Kf[b, t, h * d:(h + 1) * d]))
                                  for t in range(H * W)])
                    e = np.exp(s - s.max())
                    p = e / e.sum()
                    O[b, y, x, h * d:(h + 1) * d] = sum(p[t] * Vf[b, t, h * d:(h + 1) * d]
                                                        for t in range(H * W))
                    lse[b, h, y * W + x] = math.log(e.sum()) + s.max()
    return O, lse


def masked_attention_loops(Q, K, V, index, heads, S, scale):
    """Per query: scan the whole map, keep the tokens whose region is listed
    in the query region's index row (once per listing), softmax, weighted sum."""
    B, H, W, C = Q.shape
    d = C // heads
    O = np.zeros_like(Q)
    for b in range(B):
        for h in range(heads):
            hi = 0 if index.shape[1] == 1 else h
            for y in range(H):
                for x in range(W):
                    i = region_of(y, x, H, W, S)
                    q = Q[b, y, x, h * d:(h + 1) * d]
                    s, vals = [], []
                    for r in index[b, hi, i]:
                        for yy in range(H):
                            for xx in range(W):
                                if region_of(yy, xx, H, W, S) == r:
                                    s.append(scale * float(np.dot(q, K[b, yy, xx, h * d:(h + 1) * d])))
                                    vals.append(V[b, yy, xx, h * d:(h + 1) * d])
                    s = np.array(s)
                    p = np.exp(s - s.max())
                    p /= p.sum()
                    O[b, y, x, h * d:(h + 1) * d] = (p[:, None] * np.array(vals)).sum(axis=0)
    return O


def small_problem(seed, B=1, H=4, W=6, C=4):
    g = rng(seed)
    return (g.standard_normal((B, H, W, C)), g.standard_normal((B, H, W, C)),
            g.standard_normal((B, H, W, C)))


def test_topk_equal_S2_is_full_attention():
    """Footnote of Section 3.4: topk = S^2 means full self-attention."""
    Q, K, V = small_problem(4)
    heads, S = 2, 2
    scale = 0.37
    O, index, lse, _ = orc.bra_forward(Q, K, V, None, heads, S, S * S, scale=scale)
    Of, lsef = full_attention_loops(Q, K, V, heads, scale)
    np.testing.assert_allclose(O, Of, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, lsef, rtol=1e-11, atol=1e-12)


def test_S1_is_full_attention():
    Q, K, V = small_problem(5)
    O, index, lse, _ = orc.bra_forward(Q, K, V, None, 1, 1, 1, scale=0.5)
    assert index.shape == (1, 1, 1, 1) and index[0, 0, 0, 0] == 0
    Of, lsef = full_attention_loops(Q, K, V, 1, 0.5)
    np.testing.assert_allclose(O, Of, rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(lse, lsef, rtol=1e-11, atol=1e-12)


def test_default_scale_is_one_over_sqrt_head_dim():
    Q, K, V = small_problem(6, C=8)
    heads = 2
    O1, *_ = orc.bra_forward(Q, K, V, None, heads, 2, 2)
    O2, *_ = orc.bra_forward(Q, K, V, None, heads, 2, 2, scale=1.0 / math.sqrt(4))
    assert np.array_equal(O1, O2)


def test_routed_attention_matches_whole_map_scan():
    """Routed attention == per-query scan of the map keeping listed regions,
    for the top-k index and for a hand-made index with a duplicate."""
    Q, K, V = small_problem(7, B=2)
    heads, S, k = 2, 2, 2
    scale = 1.0 / math.sqrt(2)
    _, _, index, _ = orc.bra_route(Q, K, heads, S, k)
    O, _ = orc.bra_attend(Q, K, V, index, None, heads, S, scale)
    np.testing.assert_allclose(O, masked_attention_loops(Q, K, V, index, heads, S, scale),
                               rtol=1e-11, atol=1e-12)
    idx2 = rng(8).integers(0, S * S, size=(2, heads, S * S, 3)).astype(np.int32)
    idx2[0, 0, 0] = [3, 3, 1]          # duplicate listing counts twice
    O2, _ = orc.bra_attend(Q, K, V, idx2, None, heads, S, scale)
    np.testing.assert_allclose(O2, masked_attention_loops(Q, K, V, idx2, heads, S, scale),
                               rtol=1e-11, atol=1e-12)
    # one index shared by all heads
    idx3 = idx2[:, :1]
    O3, _ = orc.bra_attend(Q, K, V, idx3, None, heads, S, scale)
    np.testing.assert_allclose(O3, masked_attention_loops(Q, K, V, idx3, heads, S, scale),
                               rtol=1e-11, atol=1e-12)


def test_self_index_is_window_attention():
    """I[i] = {i}: every region attends within itself only."""
    Q, K, V = small_problem(9)
    S, heads = 2, 1
    R = S * S
    index = np.arange(R, dtype=np.int32).reshape(1, 1, R, 1)
    O, _ = orc.bra_attend(Q, K, V, index, None, heads, S, 1.0)
    H, W = Q.shape[1:3]
    hs, ws = H // S, W // S
    for ry in range(S):
        for rx in range(S):
            sl = (slice(0, 1), slice(ry * hs, (ry + 1) * hs), slice(rx * ws, (rx + 1) * ws))
            Ow, _ = full_attention_loops(Q[sl], K[sl], V[sl], heads, 1.0)
            np.testing.assert_allclose(O[sl], Ow, rtol=1e-11, atol=1e-12)


def test_attention_invariances():
    Q, K, V = small_problem(10, C=6)
    heads, S, k = 2, 2, 3
    _, _, index, _ = orc.bra_route(Q, K, heads, S, k)
    O, lse = orc.bra_attend(Q, K, V, index, None, heads, S)
    # permuting an index row changes nothing
    O_perm, _ = orc.bra_attend(Q, K, V, index[..., ::-1].copy(), None, heads, S)
    np.testing.assert_allclose(O_perm, O, rtol=1e-12, atol=1e-13)
    # a constant vector added to every key: softmax is shift invariant per query
    shift = rng(11).standard_normal(6)
    O_shift, _ = orc.bra_attend(Q, K + shift, V, index, None, heads, S)
    np.testing.assert_allclose(O_shift, O, rtol=1e-10, atol=1e-11)
    # constant V: rows of the softmax sum to one
    Vc = np.broadcast_to(np.arange(1.0, 7.0), V.shape).copy()
    O_const, _ = orc.bra_attend(Q, K, Vc, index, None, heads, S)
    np.testing.assert_allclose(O_const, Vc, rtol=1e-12, atol=1e-12)


def test_lse_normalises_the_scores():
    Q, K, V = small_problem(12)
    heads, S, k, scale = 1, 2, 2, 0.8
    _, _, index, _ = orc.bra_route(Q, K, heads, S, k)
    _, lse = orc.bra_attend(Q, K, V, index, None, heads, S, scale)
    B, H, W, C = Q.shape
    for y in range(H):
        for x in range(W):
            i = region_of(y, x, H, W, S)
            tot = 0.0
            for yy in range(H):
                for xx in range(W):
                    if region_of(yy, xx, H, W, S) in index[0, 0, i]:
                        tot += math.exp(scale * float(Q[0, y, x] @ K[0, yy, xx]) - lse[0, 0, y * W + x])
            assert tot == pytest.approx(1.0, abs=1e-12)


def test_out_of_range_index_is_an_error():
    Q, K, V = small_problem(13)
    bad = np.full((1, 1, 4, 1), 4, dtype=np.int32)
    with pytest.raises(IndexError):
        orc.bra_attend(Q, K, V, bad, None, 1, 2)


# ---------------------------------------------------------------- LCE
def test_lce_delta_filter_is_identity():
    V = rng(14).standard_normal((2, 5, 7, 3))
    w = np.zeros((3, 5, 5))
    w[:, 2, 2] = 1.0
    np.testing.assert_array_equal(orc.lce(V, w), V)


def test_lce_shifted_delta_picks_the_right_neighbour():
    """w[c,i,j] multiplies V[y+i-2, x+j-2]: cross-correlation orientation."""
    V = rng(15).standard_normal((1, 6, 6, 1))
    w = np.zeros((1, 5, 5))
    w[0, 0, 3] = 1.0                       # i=0 -> row y-2 ; j=3 -> column x+1
    out = orc.lce(V, w)
    for y in range(6):
        for x in range(6):
            yy, xx = y - 2, x + 1
            expect = V[0, yy, xx, 0] if 0 <= yy < 6 and 0 <= xx < 6 else 0.0
            assert out[0, y, x, 0] == expect


def test_lce_all_ones_border_sums_by_hand():
    H = W = 6
    w = rng(16).standard_normal((2, 5, 5))
    out = orc.lce(np.ones((1, H, W, 2)), w, bias=np.array([0.5, -1.0]))
    for c in range(2):
        assert out[0, 2, 3, c] == pytest.approx(w[c].sum() + (0.5, -1.0)[c])          # interior
        assert out[0, 0, 0, c] == pytest.approx(w[c, 2:, 2:].sum() + (0.5, -1.0)[c])  # corner
        assert out[0, 5, 2, c] == pytest.approx(w[c, :3, :].sum() + (0.5, -1.0)[c])   # bottom edge
        assert out[0, 1, 5, c] == pytest.approx(w[c, 1:, :3].sum() + (0.5, -1.0)[c])  # right edge, row 1


def test_lce_matches_scipy_correlate2d():
    from scipy.signal import correlate2d
    V = rng(17).standard_normal((2, 9, 8, 3))
    w = rng(18).standard_normal((3, 5, 5))
    out = orc.lce(V, w)
    for b in range(2):
        for c in range(3):
            ref = correlate2d(V[b, :, :, c], w[c], mode="same", boundary="fill", fillvalue=0.0)
            np.testing.assert_allclose(out[b, :, :, c], ref, rtol=1e-12, atol=1e-12)


def test_forward_is_attention_plus_lce():
    Q, K, V = small_problem(19, H=8, W=8)
    w = 0.1 * rng(20).standard_normal((4, 5, 5))
    heads, S, k = 2, 2, 2
    O, index, _, _ = orc.bra_forward(Q, K, V, w, heads, S, k)
    O0, index0, _, _ = orc.bra_forward(Q, K, V, np.zeros_like(w), heads, S, k)
    On, _, _, _ = orc.bra_forward(Q, K, V, None, heads, S, k)
    assert np.array_equal(index, index0)
    np.testing.assert_allclose(O0, On, rtol=0, atol=0)
    np.testing.assert_allclose(O - O0, orc.lce(V, w), rtol=1e-12, atol=1e-13)
    # LCE crosses region borders: it is a conv over the whole map, not per region
    from scipy.signal import correlate2d
    ref = correlate2d(V[0, :, :, 1], w[1], mode="same")
    np.testing.assert_allclose((O - O0)[0, :, :, 1], ref, rtol=1e-11, atol=1e-12)


# ---------------------------------------------------------------- backward
def torch_dense_reference(Q, K, V, index, w, heads, S, scale):
    """Same function through library routines: dense masked softmax attention
    (mask built from the index, duplicates as log-multiplicity) + conv2d, fp64."""
    import torch
    import torch.nn.functional as F
    B, H, W, C = Q.shape
    d = C // heads
    N = H * W
    reg = np.array([region_of(y, x, H, W, S) for y in range(H) for x in range(W)])
    mult = np.zeros((B, heads, N, N))
    for b in range(B):
        for h in range(heads):
            hi = 0 if index.shape[1] == 1 else h
            for t in range(N):
                for r in index[b, hi, reg[t]]:
                    mult[b, h, t] += (reg == r)
    logm = torch.from_numpy(np.where(mult > 0, np.log(np.maximum(mult, 1e-300)), -np.inf))
    tq, tk, tv = (torch.tensor(a, dtype=torch.float64, requires_grad=True) for a in (Q, K, V))
    tw = torch.tensor(w, dtype=torch.float64, requires_grad=True)

    def heads_first(t):
        return t.reshape(B, N, heads, d).permute(0, 2, 1, 3)
    s = scale * heads_first(tq) @ heads_first(tk).transpose(-1, -2) + logm
    o = torch.softmax(s, dim=-1) @ heads_first(tv)
    o = o.permute(0, 2, 1, 3).reshape(B, H, W, C)
    conv = F.conv2d(tv.permute(0, 3, 1, 2), tw[:, None], padding=2, groups=C).permute(0, 2, 3, 1)
    return o + conv, (tq, tk, tv, tw)


def test_forward_and_backward_match_torch_autograd_of_dense_masked_form():
    import torch
    B, H, W, C, heads, S, k = 2, 4, 4, 4, 2, 2, 3
    g = rng(21)
    Q, K, V, dO = (g.standard_normal((B, H, W, C)) for _ in range(4))
    w = 0.3 * g.standard_normal((C, 5, 5))
    index = g.integers(0, S * S, size=(B, heads, S * S, k)).astype(np.int32)
    index[1, 1, 2] = [0, 0, 3]                      # duplicate -> fan-in adds twice
    scale = 0.6
    O, _ = orc.bra_attend(Q, K, V, index, w, heads, S, scale)
    out, (tq, tk, tv, tw) = torch_dense_reference(Q, K, V, index, w, heads, S, scale)
    np.testing.assert_allclose(O, out.detach().numpy(), rtol=1e-10, atol=1e-11)
    out.backward(torch.from_numpy(dO))
    dQ, dK, dV, dw, db = orc.bra_backward(Q, K, V, index, w, dO, heads, S, scale)
    np.testing.assert_allclose(dQ, tq.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dK, tk.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dV, tv.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(dw, tw.grad.numpy(), rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(db, dO.sum(axis=(0, 1, 2)), rtol=1e-12)


def test_backward_matches_central_finite_differences():
    B, H, W, C, heads, S, k = 1, 4, 4, 2, 1, 2, 2
    g = rng(22)
    Q, K, V, dO = (g.standard_normal((B, H, W, C)) for _ in range(4))
    w = 0.3 * g.standard_normal((C, 5, 5))
    _, _, index, _ = orc.bra_route(Q, K, heads, S, k)
    scale = 0.9
    grads = orc.bra_backward(Q, K, V, index, w, dO, heads, S, scale)

    def loss(Q, K, V, w):
        O, _ = orc.bra_attend(Q, K, V, index, w, heads, S, scale)   # index frozen
        return float((O * dO).sum())
    eps = 1e-6
    args = [Q, K, V, w]
    for a_i, grad in enumerate(grads[:4]):
        flat = args[a_i].reshape(-1)
        pick = rng(23 + a_i).choice(flat.size, size=min(24, flat.size), replace=False)
        for p in pick:
            old = flat[p]
            flat[p] = old + eps
            up = loss(*args)
            flat[p] = old - eps
            dn = loss(*args)
            flat[p] = old
            assert grad.reshape(-1)[p] == pytest.approx((up - dn) / (2 * eps), rel=2e-6, abs=2e-8)


def test_backward_full_attention_case_matches_textbook_gradient():
    """topk = S^2: gradients equal those of plain softmax attention (autograd)."""
    import torch
    B, H, W, C, heads, S = 1, 4, 4, 4, 2, 2
    g = rng(30)
    Q, K, V, dO = (g.standard_normal((B, H, W, C)) for _ in range(4))
    _, _, index, _ = orc.bra_route(Q, K, heads, S, S * S)
    dQ, dK, dV, _, _ = orc.bra_backward(Q, K, V, index, None, dO, heads, S, 0.5)
    tq, tk, tv = (torch.tensor(a.reshape(B, H * W, heads, C // heads).transpose(0, 2, 1, 3),
                               requires_grad=True) for a in (Q, K, V))
    o = torch.softmax(0.5 * tq @ tk.transpose(-1, -2), -1) @ tv
    o.backward(torch.from_numpy(dO.reshape(B, H * W, heads, C // heads).transpose(0, 2, 1, 3).copy()))
    for ours, t in ((dQ, tq), (dK, tk), (dV, tv)):
        ref = t.grad.numpy().transpose(0, 2, 1, 3).reshape(B, H, W, C)
        np.testing.assert_allclose(ours, ref, rtol=1e-10, atol=1e-12)


# ---------------------------------------------------------------- maps S does not divide (Appendix C)
def hand_padded(X, S):
    """Zero padding at the bottom and right, token by token (not the oracle's slicing)."""
    B, H, W, C = X.shape
    Hp, Wp = math.ceil(H / S) * S, math.ceil(W / S) * S
    out = np.zeros((B, Hp, Wp, C))
    for b, y, x in itertools.product(range(B), range(H), range(W)):
        out[b, y, x] = X[b, y, x]
    return out


def test_pad_and_crop_place_every_token_by_hand():
    X = rng(40).standard_normal((2, 5, 7, 3))
    P = orc.pad_map(X, 3)
    assert P.shape == (2, 6, 9, 3) and orc.padded_size(5, 7, 3) == (6, 9)
    np.testing.assert_array_equal(P, hand_padded(X, 3))
    np.testing.assert_array_equal(orc.crop_map(P, 5, 7), X)
    Y = rng(41).standard_normal((1, 6, 9, 3))
    np.testing.assert_array_equal(orc.pad_map(Y, 3), Y)          # a map S divides is left alone


def test_padded_map_with_all_regions_is_full_attention_over_real_and_zero_tokens():
    """topk = S^2 on a 5 x 7 map with S = 2: every query attends to all 6 x 8 tokens of the padded map,
    the 18 zero tokens included (score 0, value 0); O and lse of the real queries equal the textbook
    routine run on hand-padded arrays, and the LCE term is the correlation of the UNPADDED V."""
    from scipy.signal import correlate2d
    B, H, W, C, heads, S = 1, 5, 7, 4, 2, 2
    g = rng(42)
    Q, K, V = (g.standard_normal((B, H, W, C)) for _ in range(3))
    w = g.standard_normal((C, 5, 5))
    scale = 0.41
    O, index, lse, _ = orc.bra_forward(Q, K, V, w, heads, S, S * S, scale=scale)
    assert O.shape == Q.shape and lse.shape == (B, heads, H * W) and index.shape == (B, heads, S * S, S * S)
    Of, lsef = full_attention_loops(hand_padded(Q, S), hand_padded(K, S), hand_padded(V, S), heads, scale)
    conv = np.stack([correlate2d(V[0, :, :, c], w[c], mode="same", boundary="fill", fillvalue=0.0)
                     for c in range(C)], axis=-1)[None]
    np.testing.assert_allclose(O, Of[:, :H, :W] + conv, rtol=1e-11, atol=1e-12)
    lse_ref = lsef.reshape(B, heads, 6, 8)[:, :, :H, :W].reshape(B, heads, H * W)
    np.testing.assert_allclose(lse, lse_ref, rtol=1e-11, atol=1e-12)


def test_padded_routing_pools_the_zero_tokens_and_matches_the_whole_map_scan():
    """Region means of a padded map divide by the full region size (zeros count); routed attention on
    the padded map equals the per-query scan over hand-padded arrays."""
    B, H, W, C, heads, S, k = 1, 5, 5, 4, 2, 3, 2
    g = rng(43)
    Q, K, V = (g.standard_normal((B, H, W, C)) for _ in range(3))
    Qr, Kr, index, _ = orc.bra_route(Q, K, heads, S, k)
    Kp = hand_padded(K, S)
    for r in range(S * S):
        ry, rx = divmod(r, S)
        np.testing.assert_allclose(Kr[0, r], Kp[0, 2 * ry:2 * ry + 2, 2 * rx:2 * rx + 2].reshape(4, C).sum(0) / 4)
    O, _ = orc.bra_attend(Q, K, V, index, None, heads, S, 0.3)
    ref = masked_attention_loops(hand_padded(Q, S), Kp, hand_padded(V, S), index, heads, S, 0.3)
    np.testing.assert_allclose(O, ref[:, :H, :W], rtol=1e-11, atol=1e-12)


def test_padded_backward_matches_central_finite_differences():
    B, H, W, C, heads, S, k = 1, 5, 7, 4, 2, 2, 2
    g = rng(44)
    Q, K, V, dO = (g.standard_normal((B, H, W, C)) for _ in range(4))
    w = 0.3 * g.standard_normal((C, 5, 5))
    _, _, index, _ = orc.bra_route(Q, K, heads, S, k)
    grads = orc.bra_backward(Q, K, V, index, w, dO, heads, S, 0.45)
    assert all(a.shape == Q.shape for a in grads[:3])

    def loss(Q, K, V, w):
        O, _ = orc.bra_attend(Q, K, V, index, w, heads, S, 0.45)
        return float((O * dO).sum())
    eps = 1e-6
    args = [Q, K, V, w]
    for a_i, grad in enumerate(grads[:4]):
        flat = args[a_i].reshape(-1)
        for p in rng(45 + a_i).choice(flat.size, size=16, replace=False):
            old = flat[p]
            flat[p] = old + eps
            up = loss(*args)
            flat[p] = old - eps
            dn = loss(*args)
            flat[p] = old
            assert grad.reshape(-1)[p] == pytest.approx((up - dn) / (2 * eps), rel=2e-6, abs=2e-8)


# ---------------------------------------------------------------- planted mistakes
def _sum_for_mean(X, S):
    return orc.region_partition(np.asarray(X, dtype=np.float64), S).sum(axis=2)


def _transposed_affinity(real):
    def f(Qr, Kr, heads, shared_routing=False):
        return real(Kr, Qr, heads, shared_routing)
    return f


def _ties_to_higher_index(real):
    def f(A, k):
        idx, gap = real(A[..., ::-1], k)
        return (A.shape[-1] - 1 - idx).astype(np.int32), gap
    return f


def _no_max_subtraction_wrong_sign(real):
    def f(Q, K, V, index, heads, S, scale):
        return real(Q, K, V, index, heads, S, -scale)
    return f


def _flipped_filter(real):
    def f(V, w, bias=None):
        return real(V, np.asarray(w)[:, ::-1, ::-1], bias)
    return f


def _replicated_border(real):
    def f(V, w, bias=None):
        V = np.asarray(V, dtype=np.float64)
        big = np.pad(V, ((0, 0), (2, 2), (2, 2), (0, 0)), mode="edge")   # edge values, not zeros, outside the map
        return real(big, w, bias)[:, 2:-2, 2:-2]
    return f


def _wrong_scale(C, heads):
    return 1.0 / np.sqrt(C)


def _dropped_lce_adjoint(real):
    def f(Q, K, V, index, w, dO, heads, S, scale=None):
        return real(Q, K, V, index, np.zeros_like(np.asarray(w, dtype=np.float64)), dO, heads, S, scale)
    return f


def _pad_at_top_left(real):
    def f(X, S):
        X = np.asarray(X, dtype=np.float64)
        Hp, Wp = orc.padded_size(X.shape[1], X.shape[2], S)
        out = np.zeros((X.shape[0], Hp, Wp, X.shape[3]))
        out[:, Hp - X.shape[1]:, Wp - X.shape[2]:] = X
        return out
    return f


PLANTED = [
    ("pad_map", _pad_at_top_left, ["test_pad_and_crop_place_every_token_by_hand",
                                   "test_padded_routing_pools_the_zero_tokens_and_matches_the_whole_map_scan"]),
    # (oracle attribute, sabotage, pins of which at least the first must fail)
    ("region_means", lambda real: _sum_for_mean, ["test_affinity_is_mean_of_all_token_pair_products"]),
    ("region_affinity", _transposed_affinity, ["test_affinity_is_mean_of_all_token_pair_products"]),
    ("topk_index", _ties_to_higher_index, ["test_topk_tie_break_lower_index_first"]),
    ("routed_attention", _no_max_subtraction_wrong_sign, ["test_topk_equal_S2_is_full_attention",
                                                          "test_S1_is_full_attention"]),
    ("default_scale", lambda real: _wrong_scale, ["test_default_scale_is_one_over_sqrt_head_dim"]),
    ("lce", _flipped_filter, ["test_lce_shifted_delta_picks_the_right_neighbour",
                              "test_lce_matches_scipy_correlate2d"]),
    ("lce", _replicated_border, ["test_lce_all_ones_border_sums_by_hand",
                                  "test_lce_matches_scipy_correlate2d"]),
    ("bra_backward", _dropped_lce_adjoint, ["test_backward_matches_central_finite_differences"]),
]


@pytest.mark.parametrize("attr,sabotage,pins", PLANTED, ids=[f"{a}-{i}" for i, (a, _, _) in enumerate(PLANTED)])
def test_pins_catch_planted_mistakes(monkeypatch, attr, sabotage, pins):
    """Plant one mistake in the oracle (a sum for the mean, a transposed operand, the wrong
    tie-break, a sign, the wrong scale, a flipped filter, a border that is not zero, a
    dropped gradient term) and run the named pins against the sabotaged oracle: each must fail."""
    for name in pins:
        globals()[name]()                               # green on the oracle as it stands
    monkeypatch.setattr(orc, attr, sabotage(getattr(orc, attr)))
    for name in pins:
        with pytest.raises((AssertionError, IndexError, ValueError)):
            globals()[name]()

"""GPU parity: the CUDA path, through the C boundary, against the fp64 CPU oracle
on the same seeded inputs.

Tolerances (stated by the benchmark definition):
  * routing index: bit-exact, except rows whose k-th and (k+1)-th oracle
    scores lie within 1e-3 relative of each other (counted and reported);
    attention is always compared using the GPU's own index
  * O: bf16 I/O max-abs <= 2e-2 and mean-abs <= 2e-3; fp32 I/O max-abs <= 1e-5
  * gradients: max-abs <= 5e-2
"""
import numpy as np
import pytest

from oracle import bra_oracle as orc
from paper_2303_08810_b200 import synthetic
from paper_2303_08810_b200.synthetic import BraConfig, CONFIGS

pytestmark = pytest.mark.gpu

TOL = {"bf16": dict(max=2e-2, mean=2e-3), "f32": dict(max=1e-5, mean=1e-6)}
GRAD_MAX = 5e-2
# d_lce_w / d_lce_b are sums over all B*H*W positions of products that are exact in fp32; with
# fp32 partial sums the rounding error is about sqrt(n) * 2^-24 of the running sum (n <= 2e5 here)
LCE_GRAD_REL = 1e-4


@pytest.fixture(scope="module")
def bra():
    import paper_2303_08810_b200 as pkg
    from paper_2303_08810_b200 import build
    build.build_library()
    pkg.load_library()
    return pkg


def to_dev(x, cfg):
    import torch
    out = {}
    for k, v in x.items():
        t = torch.from_numpy(np.ascontiguousarray(v)).cuda()
        if k != "w" and cfg.dtype == "bf16":
            t = t.to(torch.bfloat16)
        out[k] = t
    return out


def problem_of(bra, cfg, impl=0, **kw):
    return bra.make_problem(cfg.B, cfg.H, cfg.W, cfg.C, cfg.heads, cfg.S, cfg.topk, cfg.dtype,
                            impl=impl, **kw)


def f64(t):
    return t.detach().float().cpu().numpy().astype(np.float64)


def check_index(idx_gpu, idx_ref, gap, topk, R, A=None):
    """Rows whose k-th and (k+1)-th oracle scores are clearly apart must select
    exactly the oracle's regions.  The order inside a row must match too, except
    between neighbours whose oracle scores lie within 1e-3 relative (fp32 and
    fp64 may rank those either way).  Near-tie rows must still be valid."""
    clear = gap > 1e-3
    assert np.array_equal(np.sort(idx_gpu[clear], axis=-1), np.sort(idx_ref[clear], axis=-1))
    assert idx_gpu.min() >= 0 and idx_gpu.max() < R
    if topk > 1:
        assert (np.diff(np.sort(idx_gpu, axis=-1), axis=-1) > 0).all()
    order_diff = (idx_gpu != idx_ref).any(axis=-1) & clear
    if A is not None and order_diff.any():
        top = np.take_along_axis(A, idx_ref.astype(np.int64), axis=-1)     # descending scores
        rel = (top[..., :-1] - top[..., 1:]) / np.maximum(
            np.maximum(np.abs(top[..., :-1]), np.abs(top[..., 1:])), 1e-30)
        # a row may differ in order only where two neighbouring scores nearly tie
        assert (rel[order_diff].min(axis=-1) <= 1e-3).all()
        mism = idx_gpu[order_diff] != idx_ref[order_diff]
        tie = np.zeros_like(mism)
        close = rel[order_diff] <= 1e-3
        tie[:, :-1] |= close
        tie[:, 1:] |= close
        assert not (mism & ~tie).any()
    elif A is None:
        assert not order_diff.any()
    near = int((~clear).sum())
    flips = int((np.sort(idx_gpu[~clear], -1) != np.sort(idx_ref[~clear], -1)).any(axis=-1).sum()) if near else 0
    return near, flips


def oracle_affinity(x, cfg, shared=False):
    return orc.region_affinity(orc.region_means(x["Q"], cfg.S), orc.region_means(x["K"], cfg.S),
                               cfg.heads, shared)


def check_O(O_gpu, O_ref, dtype):
    err = np.abs(O_gpu - O_ref)
    assert err.max() <= TOL[dtype]["max"], f"max-abs {err.max():.3e}"
    assert err.mean() <= TOL[dtype]["mean"], f"mean-abs {err.mean():.3e}"


# ------------------------------------------------------------------ routing
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5])
def test_route_matches_oracle(bra, n):
    cfg = CONFIGS[n]
    x = synthetic.make_inputs(cfg, seed=1000 + n)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg)
    ws = bra.workspace(p)
    qm, km, idx = bra.bra_route(p, t["Q"], t["K"], ws=ws)
    assert bra.last_launch_count() >= 2
    Qr, Kr, idx_ref, gap = orc.bra_route(x["Q"], x["K"], cfg.heads, cfg.S, cfg.topk)
    np.testing.assert_allclose(f64(qm), Qr, rtol=0, atol=2e-6)
    np.testing.assert_allclose(f64(km), Kr, rtol=0, atol=2e-6)
    near, flips = check_index(idx.cpu().numpy(), idx_ref, gap, cfg.topk, cfg.R, oracle_affinity(x, cfg))
    print(f"config {n}: {near} near-tie rows of {gap.size}, {flips} differ")
    assert near < 0.02 * gap.size + 5
    assert bra.bra_device_status(ws) == 0


def test_route_shared_and_odd_shapes(bra):
    import torch
    cases = [
        (BraConfig("shared", 2, 12, 20, 48, 3, 4, 5, "f32"), True),
        (BraConfig("k=R", 1, 9, 6, 32, 2, 3, 9, "bf16"), False),
        (BraConfig("S=1", 2, 5, 7, 16, 1, 1, 1, "f32"), False),
        (BraConfig("S=16", 1, 32, 32, 32, 1, 16, 12, "bf16"), False),
        (BraConfig("R=100", 1, 20, 30, 64, 2, 10, 7, "f32"), True),
        # many winners per row and many (image, head) pairs: the thread-per-row routing kernel
        (BraConfig("k=12-many-pairs", 130, 8, 8, 64, 2, 4, 12, "bf16"), False),
        (BraConfig("k=9-shared-wide-rows", 256, 6, 6, 48, 3, 3, 9, "bf16"), True),
        # small square regions: pooled by one CTA per row of regions
        (BraConfig("1x1-regions", 3, 5, 5, 64, 2, 5, 7, "bf16"), False),
        (BraConfig("2x2-regions-f32", 2, 8, 8, 32, 1, 4, 3, "f32"), False),
        (BraConfig("4x4-regions-wide-rows", 2, 12, 12, 512, 16, 3, 2, "bf16"), True),
        # a few winners per row, many pairs, 32 channels per routing head: one CTA per (image, head)
        (BraConfig("cta-per-pair", 130, 14, 14, 64, 2, 7, 5, "bf16"), False),
        (BraConfig("cta-per-pair-k=R", 160, 4, 6, 64, 2, 2, 4, "f32"), False),
        (BraConfig("cta-per-pair-shared", 300, 6, 6, 32, 1, 3, 4, "f32"), True),
    ]
    for cfg, shared in cases:
        x = synthetic.make_inputs(cfg, seed=77)
        t = to_dev(x, cfg)
        p = problem_of(bra, cfg, shared_routing=shared)
        qm, km, idx = bra.bra_route(p, t["Q"], t["K"])
        Qr, Kr, idx_ref, gap = orc.bra_route(x["Q"], x["K"], cfg.heads, cfg.S, cfg.topk, shared)
        assert idx.shape == idx_ref.shape
        np.testing.assert_allclose(f64(qm), Qr, rtol=0, atol=2e-6)
        check_index(idx.cpu().numpy(), idx_ref, gap, cfg.topk, cfg.R, oracle_affinity(x, cfg, shared))


def test_route_exact_ties_go_to_lower_region(bra):
    """Identical K in every region: all affinities of a row are equal."""
    import torch
    cfg = BraConfig("ties", 1, 8, 8, 32, 1, 4, 3, "f32")
    Q = torch.randn(1, 8, 8, 32, device="cuda")
    K = torch.ones(1, 8, 8, 32, device="cuda")
    p = problem_of(bra, cfg)
    _, _, idx = bra.bra_route(p, Q, K)
    assert (idx.cpu().numpy() == np.array([0, 1, 2])).all()
    # +0 / -0 affinities are the same score
    Q0 = torch.zeros_like(Q)
    K0 = torch.randn_like(K)
    _, _, idx0 = bra.bra_route(p, Q0, K0)
    assert (idx0.cpu().numpy() == np.array([0, 1, 2])).all()
    # the same through the thread-per-row kernel (k > 8, many image-head pairs)
    cfg = BraConfig("ties-rows", 256, 8, 8, 32, 1, 4, 10, "f32")
    p = problem_of(bra, cfg)
    Q = torch.randn(256, 8, 8, 32, device="cuda")
    _, _, idx = bra.bra_route(p, Q, torch.ones_like(Q))
    assert (idx.cpu().numpy() == np.arange(10)).all()
    # and through the kernel with one CTA per (image, head) (2 <= k <= 8, at least 256 pairs, 32 channels per head)
    cfg = BraConfig("ties-cta-per-pair", 256, 8, 8, 32, 1, 4, 5, "f32")
    p = problem_of(bra, cfg)
    _, _, idx = bra.bra_route(p, Q, torch.ones_like(Q))
    assert (idx.cpu().numpy() == np.arange(5)).all()
    _, _, idx0 = bra.bra_route(p, torch.zeros_like(Q), torch.randn_like(Q))
    assert (idx0.cpu().numpy() == np.arange(5)).all()


# ------------------------------------------------------------------ attention
IMPLS = {"simt": 1, "mma": 2, "tc": 3, "img": 4, "auto": 0}


def run_attend_case(bra, cfg, impl, seed, shared=False, lce=True, bias=False, scale=0.0,
                    index=None, clustered=False, mutate=None):
    """One bra_attend call of kernel family `impl` against the oracle.  A family that is
    named explicitly must take the shape: BRA_ERR_UNSUPPORTED fails the test (the cases
    where a family rightly refuses a shape are asserted in
    test_kernel_families_refuse_only_what_they_should)."""
    import torch
    x = synthetic.make_inputs(cfg, seed=seed, clustered=clustered)
    if mutate is not None:
        mutate(x)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg, impl=IMPLS[impl], shared_routing=shared, lce=lce, scale=scale)
    ws = bra.workspace(p)
    if index is None:
        _, _, idx = bra.bra_route(p, t["Q"], t["K"], ws=ws)
    else:
        idx = torch.from_numpy(index).cuda()
    b = None
    b_np = None
    if bias:
        b_np = np.linspace(-0.5, 0.5, cfg.C).astype(np.float32)
        b = torch.from_numpy(b_np).cuda()
    O, lse = bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"] if lce else None, b, ws=ws)
    assert bra.last_launch_count() >= 1
    assert bra.bra_device_status(ws) == 0
    O_ref, lse_ref = orc.bra_attend(x["Q"], x["K"], x["V"], idx.cpu().numpy(),
                                    x["w"] if lce else None, cfg.heads, cfg.S,
                                    scale if scale > 0 else None, b_np)
    check_O(f64(O), O_ref, cfg.dtype)
    np.testing.assert_allclose(f64(lse), lse_ref, rtol=0, atol=1e-5 if cfg.dtype == "f32" else 2e-3)
    return O


# which benchmark configs each kernel family takes: fp32 (config 1) only the CUDA-core kernel;
# tcgen05 wants 8 x 8 or 16-wide regions (configs 2, 4); the image-resident kernel wants a head's
# K and V of a whole image in shared memory (configs 3, 5)
TAKES = {"simt": {1, 2, 3, 4, 5}, "mma": {2, 3, 4, 5}, "tc": {2, 4}, "img": {3, 5}, "auto": {1, 2, 3, 4, 5}}


@pytest.mark.parametrize("impl,n", [(i, n) for i in TAKES for n in sorted(TAKES[i])])
def test_attend_matches_oracle_on_benchmark_configs(bra, n, impl):
    run_attend_case(bra, CONFIGS[n], impl, seed=1000 + n)


@pytest.mark.parametrize("impl,n", [(i, n) for i in TAKES for n in range(1, 6) if n not in TAKES[i]])
def test_kernel_families_refuse_only_what_they_should(bra, n, impl):
    """A family asked for a shape outside its range answers BRA_ERR_UNSUPPORTED on the host,
    nothing launched; every other (family, config) pair is a parity case above."""
    import torch
    cfg = CONFIGS[n]
    x = synthetic.make_inputs(synthetic.with_batch(cfg, 1), seed=3)
    small = synthetic.with_batch(cfg, 1)
    t = to_dev(x, small)
    p = problem_of(bra, small, impl=IMPLS[impl])
    idx = torch.zeros(1, small.heads, small.R, small.topk, dtype=torch.int32, device="cuda")
    with pytest.raises(bra.BraError) as e:
        bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"])
    assert e.value.code == 7
    assert bra.last_launch_count() == 0


EDGE = [
    BraConfig("S1-n_r=90", 2, 9, 10, 32, 1, 1, 1, "f32"),
    BraConfig("rect-regions", 2, 12, 20, 64, 2, 4, 3, "bf16"),
    BraConfig("n_r=15", 1, 9, 15, 32, 2, 3, 2, "f32"),
    BraConfig("full-k=R", 1, 14, 14, 64, 2, 7, 49, "bf16"),
    BraConfig("S=1", 2, 6, 6, 32, 1, 1, 1, "bf16"),
    BraConfig("one-token-regions", 1, 4, 4, 32, 1, 4, 5, "f32"),
    BraConfig("d=64", 1, 16, 16, 128, 2, 4, 3, "bf16"),
    BraConfig("d=16", 1, 16, 16, 32, 2, 2, 2, "f32"),
    BraConfig("d=128", 1, 8, 8, 128, 1, 2, 2, "bf16"),
    BraConfig("vit-adapt-small", 1, 32, 32, 128, 2, 8, 12, "bf16"),
]


@pytest.mark.parametrize("impl", ["simt", "auto"])
@pytest.mark.parametrize("cfg", EDGE, ids=[c.name for c in EDGE])
def test_attend_edge_shapes(bra, cfg, impl):
    run_attend_case(bra, cfg, impl, seed=5)


# 8 x 8-token regions with head dim 32: the shapes of the persistent tensor-core kernel
TC_CASES = [
    BraConfig("tc-k3-two-head-pairs", 2, 32, 32, 128, 4, 4, 3, "bf16"),
    BraConfig("tc-k16-every-region", 1, 32, 32, 64, 2, 4, 16, "bf16"),
    BraConfig("tc-several-tiles-per-cta", 5, 56, 56, 64, 2, 7, 2, "bf16"),
    BraConfig("tc-single-region", 1, 8, 8, 64, 2, 1, 1, "bf16"),
    BraConfig("tc-k5-S8", 1, 64, 64, 64, 2, 8, 5, "bf16"),
]


@pytest.mark.parametrize("cfg", TC_CASES, ids=[c.name for c in TC_CASES])
def test_attend_tc_shapes(bra, cfg):
    run_attend_case(bra, cfg, "tc", seed=21)


# head dim 32, bf16, every region shape: the warp-level tensor-core kernel
MMA_CASES = TC_CASES + [
    BraConfig("mma-2x2-regions-k16", 2, 14, 14, 256, 8, 7, 16, "bf16"),
    BraConfig("mma-4x4-regions-k4", 2, 28, 28, 128, 4, 7, 4, "bf16"),
    BraConfig("mma-16x16-regions-two-chunks", 1, 32, 32, 64, 2, 2, 3, "bf16"),
    BraConfig("mma-3x5-regions-odd-width", 2, 12, 20, 64, 2, 4, 3, "bf16"),
    BraConfig("mma-last-block-partial", 1, 14, 14, 64, 2, 7, 49, "bf16"),
    BraConfig("mma-6x6-region-S1", 2, 6, 6, 32, 1, 1, 1, "bf16"),
    BraConfig("mma-7x7-regions-k3", 1, 56, 56, 64, 2, 8, 3, "bf16"),
    BraConfig("mma-one-token-regions", 1, 4, 4, 32, 1, 4, 5, "bf16"),
    BraConfig("mma-wide-regions-3-chunks", 1, 18, 64, 32, 1, 1, 1, "bf16"),
    # head dim 64: two 32-channel planes per head
    BraConfig("mma-d64-vit-adaptation", 1, 32, 32, 768, 12, 8, 12, "bf16"),
    BraConfig("mma-d64-8x8-regions-k2", 2, 16, 16, 128, 2, 2, 2, "bf16"),
    BraConfig("mma-d64-3x5-regions", 1, 12, 20, 192, 3, 4, 3, "bf16"),
    BraConfig("mma-d64-last-block-partial", 1, 14, 14, 64, 1, 7, 49, "bf16"),
]


@pytest.mark.parametrize("cfg", MMA_CASES, ids=[c.name for c in MMA_CASES])
def test_attend_mma_shapes(bra, cfg):
    run_attend_case(bra, cfg, "mma", seed=22)


def test_attend_mma_options(bra):
    cfg = BraConfig("mma-opts", 2, 16, 16, 64, 2, 4, 3, "bf16")
    run_attend_case(bra, cfg, "mma", seed=6, lce=False)
    run_attend_case(bra, cfg, "mma", seed=6, bias=True)
    run_attend_case(bra, cfg, "mma", seed=6, scale=0.5)
    run_attend_case(bra, cfg, "mma", seed=6, shared=True)
    rng = np.random.default_rng(3)
    idx = rng.integers(0, cfg.R, size=(cfg.B, cfg.heads, cfg.R, cfg.topk)).astype(np.int32)
    idx[0, 0, 0] = [5, 5, 5]
    run_attend_case(bra, cfg, "mma", seed=6, index=idx)


# head dim 32, bf16, maps small enough that one (image, head) of K and V fits in shared memory
IMG_CASES = [c for c in MMA_CASES if c.H * c.W <= 1500 and c.C // c.heads == 32] + [
    BraConfig("img-tail-tile-n_r=24", 2, 12, 16, 64, 2, 2, 3, "bf16"),
    BraConfig("img-5x5-regions-odd", 1, 15, 15, 32, 1, 3, 4, "bf16"),
    BraConfig("img-k-many-blocks", 1, 16, 16, 64, 2, 4, 16, "bf16"),
    BraConfig("img-many-images", 40, 14, 14, 64, 2, 7, 5, "bf16"),
]


@pytest.mark.parametrize("cfg", IMG_CASES, ids=[c.name for c in IMG_CASES])
def test_attend_img_shapes(bra, cfg):
    run_attend_case(bra, cfg, "img", seed=24)


def test_attend_img_options(bra):
    cfg = BraConfig("img-opts", 2, 16, 16, 64, 2, 4, 3, "bf16")
    run_attend_case(bra, cfg, "img", seed=6, lce=False)
    run_attend_case(bra, cfg, "img", seed=6, bias=True)
    run_attend_case(bra, cfg, "img", seed=6, scale=0.5)
    run_attend_case(bra, cfg, "img", seed=6, shared=True)
    run_attend_case(bra, cfg, "img", seed=6, clustered=True)
    rng = np.random.default_rng(3)
    idx = rng.integers(0, cfg.R, size=(cfg.B, cfg.heads, cfg.R, cfg.topk)).astype(np.int32)
    idx[0, 0, 0] = [5, 5, 5]
    run_attend_case(bra, cfg, "img", seed=6, index=idx)


# head dim 32, regions 16 tokens wide and a multiple of 8 high: the tcgen05 kernel for large regions
TC_WIDE_CASES = [
    BraConfig("wide-16x16-k4", 2, 32, 32, 64, 2, 2, 4, "bf16"),
    BraConfig("wide-16x16-k1-three-heads", 1, 32, 32, 96, 3, 2, 1, "bf16"),
    BraConfig("wide-8x16-regions-k3", 1, 16, 32, 32, 1, 2, 3, "bf16"),
    BraConfig("wide-24x16-regions", 1, 48, 32, 64, 2, 2, 2, "bf16"),
    BraConfig("wide-many-tiles", 3, 64, 64, 64, 2, 4, 5, "bf16"),
]


@pytest.mark.parametrize("cfg", TC_WIDE_CASES, ids=[c.name for c in TC_WIDE_CASES])
def test_attend_tc_wide_shapes(bra, cfg):
    run_attend_case(bra, cfg, "tc", seed=23)


def test_attend_tc_wide_options(bra):
    cfg = BraConfig("wide-opts", 1, 32, 32, 64, 2, 2, 2, "bf16")
    run_attend_case(bra, cfg, "tc", seed=6, lce=False)
    run_attend_case(bra, cfg, "tc", seed=6, bias=True)
    run_attend_case(bra, cfg, "tc", seed=6, scale=0.5)
    run_attend_case(bra, cfg, "tc", seed=6, shared=True)
    idx = np.array([[[[3, 3], [0, 1], [2, 0], [1, 1]]] * 2], dtype=np.int32)
    run_attend_case(bra, cfg, "tc", seed=6, index=idx)


@pytest.mark.parametrize("order", [[0, 1, 2, 3], [0, 3, 1, 2], [3, 0, 1, 2], [1, 2, 3, 3]])
@pytest.mark.parametrize("gain", [8.0, 64.0])
def test_attend_tc_wide_scores_that_grow_late(bra, order, gain):
    """The keys of one region are scaled up, so that the row maxima of its key blocks lie far above
    those of the blocks routed before it (by a few hundred at gain 64): whatever reference
    maximum the kernel carries from earlier blocks, the result must be the plain softmax."""
    cfg = BraConfig("wide-late-scores", 1, 32, 32, 64, 2, 2, 4, "bf16")

    def louder_region_3(x):
        x["K"][:, 16:, 16:, :] *= gain             # region 3 of the 2 x 2 partition

    idx = np.array([[[order] * 4] * 2], dtype=np.int32)
    run_attend_case(bra, cfg, "tc", seed=31, index=idx, mutate=louder_region_3)


OPT_CASES = [BraConfig("opts", 2, 16, 16, 64, 2, 4, 3, "bf16"),
             BraConfig("opts-8x8-regions", 2, 32, 32, 64, 2, 4, 3, "bf16")]


@pytest.mark.parametrize("cfg", OPT_CASES, ids=[c.name for c in OPT_CASES])
@pytest.mark.parametrize("impl", ["simt", "auto"])
def test_attend_options(bra, impl, cfg):
    run_attend_case(bra, cfg, impl, seed=6, lce=False)
    run_attend_case(bra, cfg, impl, seed=6, bias=True)
    run_attend_case(bra, cfg, impl, seed=6, scale=0.5)
    run_attend_case(bra, cfg, impl, seed=6, shared=True)
    run_attend_case(bra, cfg, impl, seed=6, clustered=True)
    # a caller's index: any order, duplicates count twice
    rng = np.random.default_rng(3)
    idx = rng.integers(0, cfg.R, size=(cfg.B, cfg.heads, cfg.R, cfg.topk)).astype(np.int32)
    idx[0, 0, 0] = [5, 5, 5]
    run_attend_case(bra, cfg, impl, seed=6, index=idx)


@pytest.mark.parametrize("hw", [16, 32])
@pytest.mark.parametrize("impl", ["simt", "img", "auto"])
def test_out_of_range_index_is_reported_not_fatal(bra, impl, hw):
    import torch
    cfg = BraConfig("bad-index", 1, hw, hw, 64, 2, 4, 2, "bf16")
    x = synthetic.make_inputs(cfg, seed=8)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg, impl=IMPLS[impl])
    ws = bra.workspace(p)
    idx = torch.zeros(cfg.B, cfg.heads, cfg.R, cfg.topk, dtype=torch.int32, device="cuda")
    idx[0, 1, 3, 1] = cfg.R          # one past the end
    idx[0, 0, 7, 0] = -4
    O, _ = bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 9
    assert bra.bra_device_status(ws) == 0          # cleared by the read
    assert torch.isfinite(O.float()).all()
    # the context is still usable and a clean call reports no error
    idx.zero_()
    bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 0


# ------------------------------------------------------------------ fused forward
@pytest.mark.parametrize("n", [1, 2, 3, 4, 5])
def test_forward_matches_oracle(bra, n):
    cfg = CONFIGS[n]
    x = synthetic.make_inputs(cfg, seed=1000 + n)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg)
    ws = bra.workspace(p)
    O, idx, lse = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    assert bra.last_launch_count() >= 1
    assert bra.bra_device_status(ws) == 0
    _, _, idx_ref, gap = orc.bra_route(x["Q"], x["K"], cfg.heads, cfg.S, cfg.topk)
    near, flips = check_index(idx.cpu().numpy(), idx_ref, gap, cfg.topk, cfg.R, oracle_affinity(x, cfg))
    O_ref, lse_ref = orc.bra_attend(x["Q"], x["K"], x["V"], idx.cpu().numpy(), x["w"], cfg.heads, cfg.S)
    check_O(f64(O), O_ref, cfg.dtype)
    # without the optional outputs the result is the same
    O2, _, _ = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws, want_index=False, want_lse=False)
    assert (O2 == O).all()
    print(f"config {n}: forward ok, {near} near-tie rows, {flips} differ")


def test_forward_is_deterministic(bra):
    cfg = CONFIGS[5]
    x = synthetic.make_inputs(cfg, seed=42)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg)
    ws = bra.workspace(p)
    O1, i1, l1 = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    O2, i2, l2 = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    assert (O1 == O2).all() and (i1 == i2).all() and (l1 == l2).all()


@pytest.mark.parametrize("n", [2, 3, 4, 5])
def test_forward_orders_attention_after_routing(bra, n):
    """The library's kernels overlap (programmatic dependent launch): attention must still see the
    index the routing step of the SAME call wrote.  Each call starts from an index buffer full of
    out-of-range entries and another pair of Q, K, so a kernel that read the buffer too early would
    either report a bad index or attend to the regions of the call before."""
    import torch
    cfg = CONFIGS[n]
    p = problem_of(bra, cfg)
    ws = bra.workspace(p)
    sets = [to_dev(synthetic.make_inputs(cfg, seed=77 + s), cfg) for s in range(2)]
    want = []
    for t in sets:
        _, _, idx = bra.bra_route(p, t["Q"], t["K"], ws=ws)
        O, _ = bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"], ws=ws)
        want.append((idx.clone(), O.clone()))
    assert bra.bra_device_status(ws) == 0
    idx = torch.empty_like(want[0][0])
    for it in range(6):
        t, (idx_ref, O_ref) = sets[it % 2], want[it % 2]
        idx.fill_(-7)
        O, idx, _ = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], index=idx, ws=ws)
        assert bra.bra_device_status(ws) == 0, f"call {it}"
        assert (idx == idx_ref).all() and (O == O_ref).all(), f"call {it}"


# bf16, head dim 32, 8 x 8-token regions, topk = 1, per-head routing, <= 64 regions, C <= 128: with
# BRA_IMPL_TC_FUSED bra_forward is ONE launch (pooling, routing, attention: three phases of one grid)
FUSED = 5
ONE_LAUNCH_CASES = [
    BraConfig("fused-single-region", 1, 8, 8, 64, 2, 1, 1, "bf16"),
    BraConfig("fused-one-image", 1, 56, 56, 64, 2, 7, 1, "bf16"),
    BraConfig("fused-two-head-pairs", 3, 32, 32, 128, 4, 4, 1, "bf16"),
    BraConfig("fused-64-regions", 2, 64, 64, 64, 2, 8, 1, "bf16"),
    BraConfig("fused-nine-regions", 5, 24, 24, 64, 2, 3, 1, "bf16"),
    BraConfig("fused-more-images-than-lookahead", 40, 16, 16, 64, 2, 2, 1, "bf16"),
]


@pytest.mark.parametrize("cfg", ONE_LAUNCH_CASES, ids=[c.name for c in ONE_LAUNCH_CASES])
def test_forward_in_one_launch_equals_route_then_attend(bra, cfg):
    """The one-launch forward gives, bit for bit, the index of bra_route and the O / lse of bra_attend,
    call after call on the same scratch buffer (its barrier counters clean themselves), and matches
    the oracle."""
    import torch
    p = problem_of(bra, cfg, impl=FUSED)
    ws = bra.workspace(p)
    sets = [to_dev(synthetic.make_inputs(cfg, seed=300 + s, clustered=bool(s)), cfg) for s in range(2)]
    want = []
    for t in sets:
        _, _, idx = bra.bra_route(p, t["Q"], t["K"], ws=ws)
        O, lse = bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"], ws=ws)
        want.append((idx.clone(), O.clone(), lse.clone()))
    for it in range(5):
        t, (idx_ref, O_ref, lse_ref) = sets[it % 2], want[it % 2]
        O, idx, lse = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
        assert bra.last_launch_count() == 1
        assert bra.bra_device_status(ws) == 0, f"call {it}"
        assert (idx == idx_ref).all(), f"call {it}"
        assert (O == O_ref).all() and (lse == lse_ref).all(), f"call {it}"
    x = synthetic.make_inputs(cfg, seed=300)
    _, _, idx_o, gap = orc.bra_route(x["Q"], x["K"], cfg.heads, cfg.S, cfg.topk)
    check_index(want[0][0].cpu().numpy(), idx_o, gap, cfg.topk, cfg.R, oracle_affinity(x, cfg))
    O_o, _ = orc.bra_attend(x["Q"], x["K"], x["V"], want[0][0].cpu().numpy(), x["w"], cfg.heads, cfg.S)
    check_O(f64(want[0][1]), O_o, cfg.dtype)


def test_bounded_wait_that_runs_out_is_reported_and_recoverable(bra):
    """Failure detection without a GPU fault: with the injection switch one pooled unit of the
    one-launch forward is never counted as done, so every CTA's bounded wait for the end of pooling runs
    out (no tile copy and no tensor-core work has been issued at that point), the kernel returns, and the
    status reads BRA_ERR_TIMEOUT.  Reading the status restores the scratch buffer: the next call is clean."""
    cfg = BraConfig("timeout", 3, 32, 32, 64, 2, 4, 1, "bf16")
    t = to_dev(synthetic.make_inputs(cfg, seed=9), cfg)
    p = problem_of(bra, cfg, impl=FUSED)
    ws = bra.workspace(p)
    O_ref, idx_ref, _ = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 0
    p_bad = problem_of(bra, cfg, impl=FUSED, inject=1)
    bra.bra_forward(p_bad, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 10
    assert bra.bra_device_status(ws) == 0          # cleared by the read
    for _ in range(2):
        O, idx, _ = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
        assert bra.bra_device_status(ws) == 0
        assert (O == O_ref).all() and (idx == idx_ref).all()


def test_workspace_init_makes_a_dirty_buffer_usable(bra):
    """A scratch buffer full of garbage: after bra_workspace_init an out-of-range index entry is still
    reported, and the one-launch forward (which needs its counters at zero) gives the right result."""
    import torch
    cfg = BraConfig("dirty-ws", 2, 32, 32, 64, 2, 4, 1, "bf16")
    t = to_dev(synthetic.make_inputs(cfg, seed=10), cfg)
    p = problem_of(bra, cfg, impl=FUSED)
    O_ref, idx_ref, _ = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"])
    ws = bra.workspace(p)
    ws.fill_(0xFF)
    bra.workspace_init(p, ws)
    bad = idx_ref.clone()
    bad[1, 0, 3, 0] = cfg.R
    bra.bra_attend(p, t["Q"], t["K"], t["V"], bad, t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 9
    O, idx, _ = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 0
    assert (O == O_ref).all() and (idx == idx_ref).all()


# ------------------------------------------------------------------ maps S does not divide (Appendix C)
PADDED_CASES = [
    BraConfig("pad-8x8-regions-k1", 2, 30, 29, 64, 2, 4, 1, "bf16"),          # padded to 32 x 32: tcgen05, topk = 1
    BraConfig("pad-8x8-regions-k3", 1, 61, 63, 64, 2, 8, 3, "bf16"),          # padded to 64 x 64: tcgen05, any topk
    BraConfig("pad-small-map-many-images", 40, 13, 13, 64, 2, 7, 4, "bf16"),  # padded to 14 x 14: image-resident
    BraConfig("pad-small-map", 3, 13, 14, 64, 2, 7, 4, "bf16"),               # warp-level kernel
    BraConfig("pad-wide-regions", 1, 30, 31, 64, 2, 2, 2, "bf16"),            # padded to 32 x 32, 16 x 16 regions
    BraConfig("pad-fp32", 1, 15, 14, 32, 1, 4, 2, "f32"),
]


@pytest.mark.parametrize("cfg", PADDED_CASES, ids=[c.name for c in PADDED_CASES])
def test_maps_that_S_does_not_divide(bra, cfg):
    """Forward and backward on a map zero-padded (inside the library) to the next multiples of S, against
    the oracle's padded reading: index of the padded map's regions, O / lse / gradients of the caller's size."""
    x = synthetic.make_inputs(cfg, seed=77, with_do=True)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg)
    ws = bra.workspace(p)
    O, idx, lse = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    assert bra.bra_device_status(ws) == 0
    assert tuple(O.shape) == (cfg.B, cfg.H, cfg.W, cfg.C) and tuple(lse.shape) == (cfg.B, cfg.heads, cfg.H * cfg.W)
    Qr, Kr, idx_ref, gap = orc.bra_route(x["Q"], x["K"], cfg.heads, cfg.S, cfg.topk)
    A = orc.region_affinity(Qr, Kr, cfg.heads)
    check_index(idx.cpu().numpy(), idx_ref, gap, cfg.topk, cfg.R, A)
    idn = idx.cpu().numpy()
    O_ref, lse_ref = orc.bra_attend(x["Q"], x["K"], x["V"], idn, x["w"], cfg.heads, cfg.S)
    check_O(f64(O), O_ref, cfg.dtype)
    np.testing.assert_allclose(f64(lse), lse_ref, rtol=0, atol=1e-5 if cfg.dtype == "f32" else 2e-3)
    # the two-call form gives the same
    qm, km, idx2 = bra.bra_route(p, t["Q"], t["K"], ws=ws)
    O2, lse2 = bra.bra_attend(p, t["Q"], t["K"], t["V"], idx2, t["w"], ws=ws)
    assert (idx2 == idx).all() and (O2 == O).all()
    np.testing.assert_allclose(f64(qm), Qr, rtol=0, atol=2e-6)
    g = bra.bra_backward(p, t["Q"], t["K"], t["V"], idx, t["w"], lse, t["dO"], ws=ws, want_bias_grad=True)
    assert bra.bra_device_status(ws) == 0
    ref = orc.bra_backward(x["Q"], x["K"], x["V"], idn, x["w"], x["dO"], cfg.heads, cfg.S)
    tol = GRAD_MAX if cfg.dtype == "bf16" else 2e-4
    for name, a, r in zip(("dQ", "dK", "dV", "d_lce_w", "d_lce_b"), g, ref):
        assert tuple(a.shape) == r.shape, name
        assert np.abs(f64(a) - r).max() <= tol, f"{cfg.name} {name}"


# ------------------------------------------------------------------ backward
def run_backward_case(bra, cfg, seed, clustered=False, shared=False, index=None, impl="auto"):
    import torch
    x = synthetic.make_inputs(cfg, seed=seed, with_do=True, clustered=clustered)
    t = to_dev(x, cfg)
    p = problem_of(bra, cfg, impl=IMPLS[impl], shared_routing=shared)
    ws = bra.workspace(p)
    if index is None:
        O, idx, lse = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws)
    else:
        idx = torch.from_numpy(index).cuda()
        O, lse = bra.bra_attend(p, t["Q"], t["K"], t["V"], idx, t["w"], ws=ws)
    g1 = bra.bra_backward(p, t["Q"], t["K"], t["V"], idx, t["w"], lse, t["dO"], ws=ws, want_bias_grad=True)
    assert bra.last_launch_count() >= 3
    g2 = bra.bra_backward(p, t["Q"], t["K"], t["V"], idx, t["w"], lse, t["dO"], ws=ws, want_bias_grad=True)
    assert bra.bra_device_status(ws) == 0
    for a, b in zip(g1, g2):
        assert (a == b).all(), "backward is not bit-reproducible"
    ref = orc.bra_backward(x["Q"], x["K"], x["V"], idx.cpu().numpy(), x["w"], x["dO"], cfg.heads, cfg.S)
    names = ("dQ", "dK", "dV", "d_lce_w", "d_lce_b")
    tol = GRAD_MAX if cfg.dtype == "bf16" else 2e-4
    for name, g, r in zip(names, g1, ref):
        err = np.abs(f64(g) - r).max()
        assert err <= tol, f"{cfg.name} {name}: max-abs {err:.3e}"
        if name.startswith("d_lce"):
            # sums of B*H*W exact products accumulated in fp32: besides the stated absolute
            # bound, the error stays a small fraction of the largest entry
            assert err <= LCE_GRAD_REL * max(1.0, np.abs(r).max()), f"{cfg.name} {name}: {err:.3e} rel"


def test_backward_tiny_fp32(bra):
    run_backward_case(bra, CONFIGS[1], seed=1001)


def test_backward_training_config(bra):
    run_backward_case(bra, CONFIGS[5], seed=1005)


BWD_MMA_CASES = [
    BraConfig("bwd-2x2-regions-k16", 2, 14, 14, 256, 8, 7, 16, "bf16"),
    BraConfig("bwd-8x8-regions-k2", 2, 32, 32, 64, 2, 4, 2, "bf16"),
    BraConfig("bwd-16x16-regions-multi-block", 1, 32, 32, 64, 2, 2, 3, "bf16"),
    BraConfig("bwd-last-block-partial", 1, 14, 14, 64, 2, 7, 49, "bf16"),
    BraConfig("bwd-one-token-regions", 1, 4, 4, 32, 1, 4, 5, "bf16"),
    BraConfig("bwd-3x5-regions", 2, 12, 20, 64, 2, 4, 3, "bf16"),
]


@pytest.mark.parametrize("cfg", BWD_MMA_CASES, ids=[c.name for c in BWD_MMA_CASES])
def test_backward_tensor_core_shapes(bra, cfg):
    run_backward_case(bra, cfg, seed=31)


# maps small enough for the kernels that keep a whole (image, head) slice in shared memory
BWD_IMG_CASES = [c for c in BWD_MMA_CASES if c.H * c.W <= 1500] + [
    BraConfig("bwd-img-4x4-regions-k4", 3, 28, 28, 128, 4, 7, 4, "bf16"),
    BraConfig("bwd-img-tail-tile-n_r=24", 2, 12, 16, 64, 2, 2, 3, "bf16"),
    BraConfig("bwd-img-many-images", 40, 14, 14, 64, 2, 7, 5, "bf16"),
]


@pytest.mark.parametrize("cfg", BWD_IMG_CASES, ids=[c.name for c in BWD_IMG_CASES])
def test_backward_image_resident_shapes(bra, cfg):
    run_backward_case(bra, cfg, seed=33, impl="img")


def test_backward_image_resident_options(bra):
    cfg = BraConfig("bwd-img-opts", 2, 16, 16, 64, 2, 4, 3, "bf16")
    run_backward_case(bra, cfg, seed=34, impl="img", shared=True)
    run_backward_case(bra, cfg, seed=34, impl="img", clustered=True)
    idx = np.zeros((cfg.B, cfg.heads, cfg.R, cfg.topk), dtype=np.int32)
    idx[..., 1] = np.arange(cfg.R)[None, None, :] % 5
    idx[..., 2] = 3
    run_backward_case(bra, cfg, seed=35, impl="img", index=idx)


def test_backward_tensor_core_duplicates_and_fan_in(bra):
    cfg = BraConfig("bwd-dup-bf16", 1, 8, 8, 32, 1, 2, 3, "bf16")
    idx = np.array([[[[0, 0, 3], [1, 2, 1], [3, 3, 3], [2, 0, 1]]]], dtype=np.int32)
    run_backward_case(bra, cfg, seed=12, index=idx)
    # every query region routes to region 0 (largest fan-in) and region 5 is never routed to
    cfg = BraConfig("bwd-fan-in", 2, 16, 16, 64, 2, 4, 2, "bf16")
    idx = np.zeros((cfg.B, cfg.heads, cfg.R, cfg.topk), dtype=np.int32)
    idx[..., 1] = np.arange(cfg.R)[None, None, :] % 5
    run_backward_case(bra, cfg, seed=13, index=idx)


def test_backward_edge_cases(bra):
    run_backward_case(bra, synthetic.with_batch(CONFIGS[5], 4), seed=9, clustered=True)
    run_backward_case(bra, BraConfig("bwd-shared", 2, 12, 20, 64, 2, 4, 3, "bf16"), seed=10, shared=True)
    run_backward_case(bra, BraConfig("bwd-full", 1, 8, 8, 32, 2, 2, 4, "f32"), seed=11)
    cfg = BraConfig("bwd-dup", 1, 8, 8, 32, 1, 2, 3, "f32")
    idx = np.array([[[[0, 0, 3], [1, 2, 1], [3, 3, 3], [2, 0, 1]]]], dtype=np.int32)
    run_backward_case(bra, cfg, seed=12, index=idx)


# ------------------------------------------------------------------ random shapes
@pytest.mark.parametrize("seed", [11, 12])
def test_random_shapes_forward_and_backward(bra, seed):
    """Seeded random problems (head dim 32, bf16): region shapes from 1 x 1 to 8 x 8 and 16-wide, any S in
    {1, 2, 3, 4, 7}, 1-4 heads, k up to 12, every kernel family that accepts the shape, per-head and
    shared routing.  Forward against the oracle on the GPU's own index, then every gradient."""
    rng = np.random.default_rng(seed)
    ran = 0
    for it in range(16):
        S = int(rng.choice([1, 2, 3, 4, 7]))
        hs, ws = int(rng.integers(1, 9)), int(rng.integers(1, 9))
        if rng.random() < 0.3:
            ws, hs = 16, 8 * int(rng.integers(1, 3))
        heads = int(rng.choice([1, 2, 3, 4]))
        B = int(rng.choice([1, 2, 3, 40]))
        if B == 40 and S * S * hs * ws > 300:
            B = 3
        k = int(rng.integers(1, min(S * S, 12) + 1))
        cfg = BraConfig(f"rnd{seed}-{it}", B, S * hs, S * ws, 32 * heads, heads, S, k, "bf16")
        impl = str(rng.choice(["auto", "img", "mma", "tc"]))
        shared = bool(rng.random() < 0.2)
        x = synthetic.make_inputs(cfg, seed=100 * seed + it, with_do=True)
        t = to_dev(x, cfg)
        p = problem_of(bra, cfg, impl=IMPLS[impl], shared_routing=shared)
        ws_buf = bra.workspace(p)
        try:
            O, idx, lse = bra.bra_forward(p, t["Q"], t["K"], t["V"], t["w"], ws=ws_buf)
        except bra.BraError as e:
            assert e.code == 7 and impl != "auto"        # that kernel family does not take the shape
            continue
        assert bra.bra_device_status(ws_buf) == 0
        idn = idx.cpu().numpy()
        O_ref, lse_ref = orc.bra_attend(x["Q"], x["K"], x["V"], idn, x["w"], cfg.heads, cfg.S)
        check_O(f64(O), O_ref, cfg.dtype)
        np.testing.assert_allclose(f64(lse), lse_ref, rtol=0, atol=2e-3)
        g = bra.bra_backward(p, t["Q"], t["K"], t["V"], idx, t["w"], lse, t["dO"], ws=ws_buf, want_bias_grad=True)
        assert bra.bra_device_status(ws_buf) == 0
        ref = orc.bra_backward(x["Q"], x["K"], x["V"], idn, x["w"], x["dO"], cfg.heads, cfg.S)
        for name, a, r in zip(("dQ", "dK", "dV", "d_lce_w", "d_lce_b"), g, ref):
            assert np.abs(f64(a) - r).max() <= GRAD_MAX, f"{cfg} {impl} {name}"
        ran += 1
    assert ran >= 8

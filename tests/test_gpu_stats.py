"""Parity of the CUDA statistics path with the CPU oracle, element by element, through the C ABI.

Tolerances (relative, against the oracle evaluated on the same rounded inputs):
  fp32 inputs 1e-5, bf16 inputs 1e-3 on gbar_sq, var_norm, var_ip, sum_sq, each relative to itself.
  var_orth is evaluated on the GPU as var_norm - var_ip / N.  Where the orthogonality ratio
  var_orth / (nu^2 N) is the larger of the augmented test's two ratios (theta = nu), i.e. where it
  decides T, var_orth must hold the tolerance relative to itself; elsewhere (var_orth is the small
  difference of two larger numbers and does not decide) its error is bounded by tol * var_norm.
  Batch sizes are compared bit-exactly unless the deciding ratio lies within tol of an integer.
"""
import math

import numpy as np
import pytest
import torch

import oracle.abs_oracle as orc
import paper_2406_13936_b200 as pkg
from paper_2406_13936_b200 import inputs

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-5, torch.bfloat16: 1e-3}


@pytest.fixture(scope="module")
def ctx():
    c = pkg.Context(0)
    yield c
    c.close()


def to_f64(G):
    """Host fp64 copy of a device tensor, exact for fp32 and bf16."""
    if G.dtype == torch.bfloat16:
        shape = G.shape
        return orc.bf16_bits_to_f64(inputs.bf16_bits(G)).reshape(shape)
    return G.detach().cpu().numpy().astype(np.float64)


def check_record(rec, ref, tol, b):
    assert rec["rows"] == b
    assert rec["status"] == ref["status"]
    assert rec["gbar_sq"] == pytest.approx(ref["gbar_sq"], rel=tol)
    assert rec["var_norm"] == pytest.approx(ref["var_norm"], rel=tol, abs=1e-300)
    assert rec["var_ip"] == pytest.approx(ref["var_ip"], rel=tol, abs=1e-300)
    N = ref["gbar_sq"]
    orth_decides = ref["var_orth"] * N >= ref["var_ip"]          # theta == nu: compare var_orth/N with var_ip/N^2
    bound = tol * (ref["var_orth"] if orth_decides else ref["var_norm"])
    assert abs(rec["var_orth"] - ref["var_orth"]) <= bound + 1e-300
    assert rec["sum_sq"] == pytest.approx(ref["sum_sq"], rel=tol)


def run_gpu(ctx, G, want_gbar=True):
    M, b, d = G.shape
    stats = ctx.new_stats(M)
    gbar = torch.full((M, d), float("nan"), device=G.device, dtype=torch.float32) if want_gbar else None
    ctx.abs_test_stats(G, stats, gbar)
    torch.cuda.synchronize()
    return pkg.stats_to_dicts(stats), gbar


def make_G(seed, M, b, d, dtype, sigma=1.0, pad=0, offset=0):
    """Gaussian-recipe rows on the GPU, optionally inside a padded / offset buffer."""
    base = inputs.gaussian_rows(seed, M, b, d, sigma, device="cpu").to("cuda")
    base = base.to(dtype)
    if pad == 0 and offset == 0:
        return base
    buf = torch.zeros(M * b * (d + pad) + offset + 64, device="cuda", dtype=dtype)
    view = buf[offset:offset + M * b * (d + pad)].view(M, b, d + pad)[:, :, :d]
    view.copy_(base)
    return view


SHAPES = [
    # (M, b, d) spanning one to several tiles, ragged tails, every tile shape the chooser has
    (1, 2, 1), (1, 2, 5), (1, 3, 8), (2, 5, 131), (1, 16, 1000), (3, 16, 4099), (1, 17, 2048),
    (1, 33, 3000), (2, 64, 2500), (1, 100, 1531), (1, 128, 5000), (1, 129, 777), (1, 256, 4099),
    (1, 257, 1200), (1, 300, 900), (1, 512, 1100), (1, 1000, 515), (1, 1024, 700), (1, 2048, 300),
    (1, 4096, 130), (8, 16, 20000), (1, 64, 70001),
    # fewer than 8 rows: several boxes per copy (segment map when d is a multiple of 256, else pairs)
    (1, 2, 256), (2, 3, 1024), (1, 4, 70144), (3, 7, 2560), (1, 5, 256000), (1, 4, 1000), (2, 6, 4104), (8, 2, 51200),
]


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("M,b,d", SHAPES)
def test_stats_match_oracle_aligned(ctx, M, b, d, dtype):
    pad = (-d) % (4 if dtype == torch.float32 else 8)      # keep the rows 16-byte aligned: tiled kernel
    G = make_G(1000 + b + d, M, b, d, dtype, sigma=1.0, pad=pad)
    recs, gbar = run_gpu(ctx, G)
    H = to_f64(G)
    for m in range(M):
        ref = orc.batch_test_stats(H[m])
        check_record(recs[m], ref, TOL[dtype], b)
        scale = np.abs(ref["gbar"]).max()
        np.testing.assert_allclose(gbar[m].cpu().numpy(), ref["gbar"], rtol=1e-5, atol=1e-6 * scale)


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("M,b,d,pad,offset", [(1, 2, 1, 0, 1), (2, 7, 333, 1, 0), (1, 64, 1001, 0, 0),
                                              (2, 19, 1030, 3, 1), (1, 300, 515, 0, 1), (1, 5000, 40, 0, 0)])
def test_stats_match_oracle_unaligned(ctx, M, b, d, pad, offset, dtype):
    G = make_G(2000 + b + d, M, b, d, dtype, sigma=3.0, pad=pad, offset=offset)
    recs, gbar = run_gpu(ctx, G)
    H = to_f64(G)
    for m in range(M):
        ref = orc.batch_test_stats(H[m])
        check_record(recs[m], ref, TOL[dtype], b)
        np.testing.assert_allclose(gbar[m].cpu().numpy(), ref["gbar"], rtol=1e-5,
                                   atol=1e-6 * np.abs(ref["gbar"]).max())


@pytest.mark.parametrize("sigma", [0.1, 1.0, 10.0])
@pytest.mark.parametrize("b,d", [(64, 100000), (256, 30000)])
def test_stats_sigma_sweep(ctx, b, d, sigma):
    G = make_G(3000 + b, 1, b, d, torch.float32, sigma=sigma)
    recs, _ = run_gpu(ctx, G, want_gbar=False)
    check_record(recs[0], orc.batch_test_stats(to_f64(G)[0]), 1e-5, b)


def test_heavy_tailed_bf16_rows(ctx):
    G = inputs.student_t_rows(7, 2, 16, 50000, device="cpu").to("cuda")
    recs, _ = run_gpu(ctx, G, want_gbar=False)
    H = to_f64(G)
    for m in range(2):
        check_record(recs[m], orc.batch_test_stats(H[m]), 1e-3, 16)


def test_tiled_and_generic_kernels_agree_and_are_deterministic(ctx):
    G = make_G(5, 2, 48, 9000, torch.float32)
    a, ga = run_gpu(ctx, G)
    a2, ga2 = run_gpu(ctx, G)
    assert a == a2 and torch.equal(ga, ga2)                 # bit-identical repeat
    ctx.set_tuning("stats_force_generic", 1)
    try:
        g, gg = run_gpu(ctx, G)
    finally:
        ctx.set_tuning("stats_force_generic", 0)
    for ra, rg in zip(a, g):
        for key in ("gbar_sq", "var_norm", "var_ip", "var_orth", "sum_sq"):
            assert ra[key] == pytest.approx(rg[key], rel=1e-6)
    np.testing.assert_allclose(ga.cpu().numpy(), gg.cpu().numpy(), rtol=1e-6, atol=1e-6 * ga.abs().max().item())


@pytest.mark.parametrize("M,b,d", [(1, 16, 9000), (2, 7, 3001), (3, 32, 5000), (1, 24, 700), (1, 2, 40)])
def test_gram_and_tiled_kernels_agree_on_bf16(ctx, M, b, d):
    """bf16 input with b <= 32 goes through the tensor-core Gram kernel; the tiled kernel must give
    the same statistics (and both match the oracle) when the Gram kernel is switched off."""
    G = make_G(70 + b, M, b, d + (-d) % 8, torch.bfloat16, sigma=2.0)
    gram, gbar_g = run_gpu(ctx, G)
    ctx.set_tuning("stats_no_gram", 1)
    try:
        tiled, gbar_t = run_gpu(ctx, G)
    finally:
        ctx.set_tuning("stats_no_gram", 0)
    H = to_f64(G)
    for m in range(M):
        ref = orc.batch_test_stats(H[m])
        check_record(gram[m], ref, 1e-3, b)
        check_record(tiled[m], ref, 1e-3, b)
        # the Gram kernel adds exact products: it is far inside the bf16 tolerance
        for key in ("gbar_sq", "var_norm", "sum_sq"):
            assert gram[m][key] == pytest.approx(ref[key], rel=1e-5)
    np.testing.assert_allclose(gbar_g.cpu().numpy(), gbar_t.cpu().numpy(), rtol=1e-6,
                               atol=1e-6 * gbar_t.abs().max().item())


@pytest.mark.parametrize("want_gbar", [False, True])
@pytest.mark.parametrize("M,b,d,pad", [(1, 33, 2048, 0), (2, 40, 5003, 5), (1, 64, 9000, 0), (3, 100, 4104, 0),
                                       (1, 128, 8200, 8), (1, 96, 300, 4), (1, 128, 300000, 0), (2, 72, 150001, 7),
                                       (1, 48, 256, 0), (1, 127, 1025, 7), (1, 50, 1, 7), (1, 33, 8, 0),
                                       (4, 128, 40000, 0), (1, 65, 2000, 0), (5, 41, 7777, 7),
                                       (1, 129, 3000, 0), (2, 136, 5003, 5), (1, 160, 40000, 0), (1, 192, 9000, 0),
                                       (1, 200, 70001, 7), (3, 255, 2049, 7), (1, 256, 100000, 0), (1, 256, 128, 0)])
def test_tcgen05_gram_kernel_matches_oracle_and_tiled_kernel(ctx, M, b, d, pad, want_gbar):
    """bf16 input with 32 < b <= 256 and 16-byte aligned rows goes through the tcgen05 Gram kernel
    (with and without the column-mean warps); the tiled kernel must give the same statistics, and
    both must match the oracle, also with a ragged last tile and a last 16-byte chunk cut by d."""
    assert pkg.plan_stats("bf16", b)["route"] == 4
    G = make_G(170 + b, M, b, d, torch.bfloat16, sigma=2.0, pad=pad)
    assert (G.stride(1) * 2) % 16 == 0 and G.data_ptr() % 16 == 0
    tc, gbar_tc = run_gpu(ctx, G, want_gbar)
    again, _ = run_gpu(ctx, G, want_gbar)
    assert again == tc                                      # fixed order of additions: bit-identical records
    ctx.set_tuning("stats_no_gram", 1)
    try:
        tiled, gbar_t = run_gpu(ctx, G, want_gbar)
    finally:
        ctx.set_tuning("stats_no_gram", 0)
    H = to_f64(G)
    for m in range(M):
        ref = orc.batch_test_stats(H[m])
        check_record(tc[m], ref, 1e-3, b)
        check_record(tiled[m], ref, 1e-3, b)
        for key in ("gbar_sq", "var_norm", "sum_sq"):
            assert tc[m][key] == pytest.approx(ref[key], rel=1e-5)
    if want_gbar:
        np.testing.assert_allclose(gbar_tc.cpu().numpy(), H.mean(axis=1), rtol=1e-5,
                                   atol=1e-6 * float(np.abs(H).max()))
        np.testing.assert_allclose(gbar_tc.cpu().numpy(), gbar_t.cpu().numpy(), rtol=1e-6,
                                   atol=1e-6 * gbar_t.abs().max().item())


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("M,b,d", [(1, 512, 3000), (2, 700, 1300), (1, 1024, 2100), (1, 1500, 640), (1, 2048, 520),
                                   (1, 3000, 200), (1, 4096, 264)])
def test_cluster_and_tiled_kernels_agree(ctx, M, b, d, dtype):
    """b > 256 splits the rows over a thread-block cluster; with that switched off the single-CTA
    tiled kernel takes the call.  Both must match the oracle and each other."""
    G = make_G(90 + b, M, b, d + (-d) % 8, dtype, sigma=1.5)
    clus, gbar_c = run_gpu(ctx, G)
    ctx.set_tuning("stats_no_cluster", 1)
    try:
        tiled, gbar_t = run_gpu(ctx, G)
    finally:
        ctx.set_tuning("stats_no_cluster", 0)
    H = to_f64(G)
    for m in range(M):
        ref = orc.batch_test_stats(H[m])
        check_record(clus[m], ref, TOL[dtype], b)
        check_record(tiled[m], ref, TOL[dtype], b)
    np.testing.assert_allclose(gbar_c.cpu().numpy(), gbar_t.cpu().numpy(), rtol=1e-6,
                               atol=1e-6 * gbar_t.abs().max().item())
    again, _ = run_gpu(ctx, G)
    assert again == clus                                     # fixed reduction order


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("b,d", [(513, 520), (514, 264), (1026, 392), (2049, 136), (769, 300), (4095, 72)])
def test_cluster_whose_last_cta_is_several_row_groups_short(ctx, b, d, dtype):
    """With RC = ceil(b/C) rows per CTA the cluster's last CTA holds b - (C-1)*RC rows, which can be
    more than one row group short of RC (b = 513, C = 4: 126 of 129).  Rows past the batch are
    zero-filled by the tile loads and must not enter the centred sums: a row of zeros that counted
    would add ||gbar||^2 to the variance, which small noise (sigma = 0.1) makes visible, and identical
    rows must still give exactly zero variance."""
    assert pkg.plan_stats("f32" if dtype == torch.float32 else "bf16", b)["route"] == 1
    G = make_G(95 + b, 1, b, d, dtype, sigma=0.1)
    recs, gbar = run_gpu(ctx, G)
    ref = orc.batch_test_stats(to_f64(G)[0])
    check_record(recs[0], ref, TOL[dtype], b)
    np.testing.assert_allclose(gbar[0].cpu().numpy(), ref["gbar"], rtol=1e-5, atol=1e-6 * np.abs(ref["gbar"]).max())
    same = G[:, :1].expand(1, b, d).contiguous()
    rec = run_gpu(ctx, same, want_gbar=False)[0][0]
    assert rec["status"] == 0 and rec["gbar_sq"] > 0
    assert rec["var_norm"] <= 1e-10 * rec["gbar_sq"] and rec["var_ip"] <= 1e-10 * rec["gbar_sq"] ** 2


@pytest.mark.parametrize("key,value", [("stats_stages", 2), ("stats_stages", 6), ("stats_stage_kb", 16),
                                       ("stats_flush_every", 1), ("stats_ctas_per_worker", 3)])
def test_tuning_knobs_do_not_change_the_result(ctx, key, value):
    G = make_G(6, 1, 200, 6000, torch.float32)
    ref = orc.batch_test_stats(to_f64(G)[0])
    ctx.set_tuning(key, value)
    try:
        recs, _ = run_gpu(ctx, G, want_gbar=False)
    finally:
        ctx.set_tuning(key, 0)
    check_record(recs[0], ref, 1e-5, 200)


def test_degenerate_inputs(ctx):
    row = torch.randn(1000, generator=torch.Generator().manual_seed(0))
    same = row.repeat(8, 1).unsqueeze(0).cuda()
    rec = run_gpu(ctx, same, want_gbar=False)[0][0]
    assert rec["status"] == 0
    assert rec["var_norm"] <= 1e-12 * rec["gbar_sq"] and rec["var_ip"] <= 1e-12 * rec["gbar_sq"] ** 2
    zero = torch.zeros((1, 4, 100), device="cuda")
    rec = run_gpu(ctx, zero, want_gbar=False)[0][0]
    assert rec["status"] == orc.STATUS_ZERO_MEAN and rec["var_norm"] == 0.0 and rec["gbar_sq"] == 0.0
    anti = torch.tensor([[[1.0, -2.0], [-1.0, 2.0]]], device="cuda")
    rec = run_gpu(ctx, anti, want_gbar=False)[0][0]
    assert rec["status"] == orc.STATUS_ZERO_MEAN and rec["var_norm"] == 10.0 and rec["var_orth"] == 10.0
    bad = torch.ones((2, 4, 64), device="cuda")
    bad[1, 2, 17] = float("inf")
    recs = run_gpu(ctx, bad, want_gbar=False)[0]
    assert recs[0]["status"] == 0 and recs[1]["status"] & orc.STATUS_NONFINITE
    nan = torch.ones((1, 4, 64), device="cuda")
    nan[0, 0, 0] = float("nan")
    assert run_gpu(ctx, nan, want_gbar=False)[0][0]["status"] & orc.STATUS_NONFINITE


@pytest.mark.parametrize("b,d,pad", [(4096, 255, 0), (4096, 256, 0), (3000, 65, 1), (3000, 64, 0), (1500, 257, 3), (700, 1000, 0)])
def test_long_columns_do_not_wear_the_low_bits_away(ctx, b, d, pad):
    """Thousands of rows whose terms all round the same way: one entry of 3 among zeros (every later
    term of the centred sum of squares is below half an ulp of the running sum), and identical rows
    (a mean that is off by the rounding of a long fp32 sum shows up as variance).  Both the aligned
    route and the alignment-free kernel must keep their fp32 chains short."""
    base = torch.zeros((1, b, d))
    base[0, 5, d // 2] = 3.0
    G = make_G(0, 1, b, d, torch.float32, pad=pad)
    G.copy_(base.to("cuda"))
    rec = run_gpu(ctx, G, want_gbar=False)[0][0]
    ref = orc.batch_test_stats(base[0].double().numpy())
    assert rec["sum_sq"] == pytest.approx(9.0, rel=1e-5)
    assert rec["var_norm"] == pytest.approx(ref["var_norm"], rel=1e-5)
    assert rec["gbar_sq"] == pytest.approx(ref["gbar_sq"], rel=1e-5)
    row = torch.randn(d, generator=torch.Generator().manual_seed(1))
    G.copy_(row.repeat(b, 1).unsqueeze(0).to("cuda"))
    rec = run_gpu(ctx, G, want_gbar=False)[0][0]
    assert rec["status"] == 0
    assert rec["gbar_sq"] == pytest.approx(float(row.double().pow(2).sum()), rel=1e-5)
    assert rec["var_norm"] <= 1e-11 * rec["gbar_sq"]


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_randomised_shapes_strides_and_recipes_against_the_oracle(ctx, seed):
    """Seeded random cases: M, b (around every tile and cluster boundary), d, row padding and base offset
    (aligned and not), both types, with or without gbar, five input recipes; every record is compared
    with the oracle.  (Single-column cases are left out: with d = 1 and a mean far below the noise,
    N itself is ill-conditioned in fp32.)"""
    import random
    rng = random.Random(seed)
    for case in range(60):
        dtype = rng.choice([torch.float32, torch.bfloat16])
        M = rng.choice([1, 1, 2, 3, 8])
        b = rng.choice([2, 3, 5, 8, 9, 16, 17, 32, 33, 40, 41, 64, 65, 128, 129, 136, 192, 256, 257, 300, 512, 513,
                        1000, 1024, 1025, 1500, 2048, 2049, 3000, 4096, rng.randint(2, 4096)])
        dmax = max(2, 400_000 // (M * b))
        d = min(dmax, rng.choice([2, 3, 7, 8, 63, 64, 65, 255, 256, 257, 1000, 4099, rng.randint(2, dmax)]))
        align = 4 if dtype == torch.float32 else 8
        pad = rng.choice([0, 0, align, 3 * align, 1, 3, 5])
        offset = rng.choice([0, 0, align, 1, 2, 3])
        recipe = rng.choice(["noise", "noise", "mean", "t", "onehot"])
        g = torch.Generator("cpu").manual_seed(1000 * seed + case)
        if recipe == "noise":
            base = torch.randn((1, 1, d), generator=g) / math.sqrt(d) + rng.choice([0.1, 1.0, 10.0]) * torch.randn((M, b, d), generator=g)
        elif recipe == "mean":
            base = torch.randn((1, 1, d), generator=g) + rng.choice([1e-3, 1e-2, 0.1]) * torch.randn((M, b, d), generator=g)
        elif recipe == "t":
            chi = torch.randn((3, M, b, d), generator=g).pow(2).sum(0) / 3
            base = 1e-3 * torch.randn((M, b, d), generator=g) / chi.sqrt() + 1e-4
        else:
            base = torch.zeros((M, b, d))
            base[:, rng.randrange(b), rng.randrange(d)] = 3.0
        base = base.to(dtype)
        buf = torch.zeros(M * b * (d + pad) + offset + 64, device="cuda", dtype=dtype)
        G = buf[offset:offset + M * b * (d + pad)].view(M, b, d + pad)[:, :, :d]
        G.copy_(base.to("cuda"))
        want_gbar = rng.random() < 0.5
        recs, gbar = run_gpu(ctx, G, want_gbar=want_gbar)
        tol = 1e-5 if dtype == torch.float32 else 1e-3
        what = (seed, case, dtype, M, b, d, pad, offset, recipe)
        for m in range(M):
            G64 = base[m].to(torch.float64).numpy()
            ref = orc.batch_test_stats(G64)
            rec = recs[m]
            assert rec["rows"] == b and rec["status"] == ref["status"], what
            assert rec["gbar_sq"] == pytest.approx(ref["gbar_sq"], rel=tol), what
            assert rec["var_norm"] == pytest.approx(ref["var_norm"], rel=tol), what
            assert rec["sum_sq"] == pytest.approx(ref["sum_sq"], rel=tol), what
            N = ref["gbar_sq"]
            # V_ip enters the test as V_ip / N^2 beside V_orth / N: where it is far below N V_norm its own
            # digits do not matter, the bound is then relative to that scale
            assert abs(rec["var_ip"] - ref["var_ip"]) <= max(tol * ref["var_ip"], tol * 1e-3 * N * ref["var_norm"]), what
            orth_decides = ref["var_orth"] * N >= ref["var_ip"]
            assert abs(rec["var_orth"] - ref["var_orth"]) <= tol * (ref["var_orth"] if orth_decides else ref["var_norm"]), what
            if want_gbar:
                err = np.abs(gbar[m].double().cpu().numpy() - G64.mean(axis=0)).max()
                assert err <= 2e-6 * np.abs(G64).max(), what


def test_contexts_and_the_context_free_call_do_not_shrink_each_other_s_kernels(ctx):
    """The shared-memory size a kernel may be launched with is a property of the kernel in the process,
    not of a context.  Different batch sizes run the same kernel with different tile buffers: a second
    context, or the context-free entry point, that needs a smaller one must not leave the first context
    (which remembers what it was granted) unable to launch the larger one."""
    other = pkg.Context(0)
    try:
        # (33, 257): without a context 257 rows go to the tiled kernel too, with the shape 33 rows use
        for b_big, b_small in ((33, 257), (60, 33), (15, 9), (250, 130), (1000, 600), (4000, 2100)):
            big = make_G(50 + b_big, 1, b_big, 20000, torch.float32)
            small = make_G(60 + b_small, 1, b_small, 20000, torch.float32)
            ref = run_gpu(ctx, big)[0][0]
            st = ctx.new_stats(1)
            other.abs_test_stats(small, st)
            if b_small <= 2048:
                pkg.abs_test_stats_noalloc(small, st)
            torch.cuda.synchronize()
            again = run_gpu(ctx, big)[0][0]
            assert again == ref
            other.abs_test_stats(big, st)
            torch.cuda.synchronize()
            assert pkg.stats_to_dicts(st)[0] == ref
    finally:
        other.close()


def test_invalid_arguments_are_rejected_before_any_launch(ctx):
    G = torch.ones((1, 1, 16), device="cuda")
    with pytest.raises(pkg.AbsError, match="b must be >= 2"):
        ctx.abs_test_stats(G, ctx.new_stats(1))
    with pytest.raises(pkg.AbsError):
        ctx.abs_test_stats(torch.ones((1, 4, 16), device="cuda", dtype=torch.float16), ctx.new_stats(1))
    with pytest.raises(pkg.AbsError, match="unknown tuning key"):
        ctx.set_tuning("no_such_knob", 1)


def test_host_entry_point_matches_device_entry_point(ctx):
    G = inputs.gaussian_rows(11, 2, 32, 5000, 1.0, device="cpu")
    recs_h, gbar_h = ctx.abs_test_stats_host(G.pin_memory(), want_gbar=True)
    recs_d, gbar_d = run_gpu(ctx, G.cuda())
    assert recs_h == recs_d
    assert torch.equal(gbar_h, gbar_d.cpu())
    Gb = G.to(torch.bfloat16)
    recs_h, _ = ctx.abs_test_stats_host(Gb)
    assert recs_h == run_gpu(ctx, Gb.cuda(), want_gbar=False)[0]


# ------------------------------------------------------------------ next batch size
def _near_boundary(ratio, tol):
    return abs(ratio - round(ratio)) <= tol * max(ratio, 1.0)


@pytest.mark.parametrize("kind,cfg", [("norm", dict(eta=0.5)), ("aug_ip", dict(theta=0.5, nu=0.5)),
                                      ("norm", dict(eta=0.9, row_weight=4.0, divisor=3.0))])
@pytest.mark.parametrize("M,b,d,sigma", [(1, 16, 3000, 1.0), (4, 16, 2000, 0.05), (8, 64, 1500, 10.0), (3, 5, 400, 0.3)])
def test_next_batch_matches_oracle(ctx, kind, cfg, M, b, d, sigma):
    G = make_G(4000 + b + M, M, b, d, torch.float32, sigma=sigma)
    stats = ctx.new_stats(M)
    ctx.abs_test_stats(G, stats)
    b_cur = torch.tensor([b], dtype=torch.int64, device="cuda")
    b_next = torch.zeros(1, dtype=torch.int64, device="cuda")
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    for b_max in (10 ** 6, b + 3):
        ctx.abs_next_batch(stats, pkg.make_test_cfg(kind, b_max, **cfg), b_cur, b_next, T_out)
        torch.cuda.synchronize()
        # (i) integer logic: the oracle applied to the GPU's own records must agree bit for bit
        recs = pkg.stats_to_dicts(stats)
        exp_b, exp_T = orc.next_batch(recs, b, b_max, kind, **cfg)
        assert T_out.tolist() == exp_T and b_next.item() == exp_b
        # (ii) end to end against the oracle's statistics, bit-exact away from rounding boundaries
        H = to_f64(G)
        refs = [orc.batch_test_stats(H[m]) for m in range(M)]
        ref_b, ref_T = orc.next_batch(refs, b, b_max, kind, **cfg)
        scale = cfg.get("row_weight", 1.0) / cfg.get("divisor", 1.0)
        for m in range(M):
            N = refs[m]["gbar_sq"]
            if kind == "norm":
                ratios = [scale * refs[m]["var_norm"] / (cfg["eta"] ** 2 * N)]
            else:
                ratios = [scale * refs[m]["var_ip"] / (cfg["theta"] ** 2 * N * N),
                          scale * refs[m]["var_orth"] / (cfg["nu"] ** 2 * N)]
            if not any(_near_boundary(r, 1e-5) for r in ratios):
                assert T_out[m].item() == ref_T[m]
            else:
                assert abs(T_out[m].item() - ref_T[m]) <= 1
        if T_out.tolist() == ref_T:
            assert b_next.item() == ref_b


def test_next_batch_edge_cases(ctx):
    stats = ctx.new_stats(3)
    host = np.zeros((3, 7))
    host[0, :5] = [0.0, 2.5, 0.0, 2.5, 5.0]      # N == 0 with variance: ratio is +inf
    host[1, :5] = [1.0, 1e300, 0.0, 0.0, 0.0]    # huge but finite ratio
    host[2, :5] = [1.0, 0.3, 0.0, 0.0, 0.0]
    as_int = host.view(np.int64)
    as_int[:, 5] = 4
    as_int[0, 6] = orc.STATUS_ZERO_MEAN
    stats.copy_(torch.from_numpy(host))
    b_cur = torch.tensor([4], dtype=torch.int64, device="cuda")
    b_next = torch.zeros(1, dtype=torch.int64, device="cuda")
    T_out = torch.zeros(3, dtype=torch.int64, device="cuda")
    ctx.abs_next_batch(stats, pkg.make_test_cfg("norm", 512, eta=0.5), b_cur, b_next, T_out)
    assert T_out.tolist() == [orc.T_SATURATE, orc.T_SATURATE, 2] and b_next.item() == 512
    as_int[0, 6] = orc.STATUS_NONFINITE          # flagged records give no decision
    as_int[1, 6] = orc.STATUS_NONFINITE
    stats.copy_(torch.from_numpy(host))
    ctx.abs_next_batch(stats, pkg.make_test_cfg("norm", 512, eta=0.5), b_cur, b_next, T_out)
    assert T_out.tolist() == [0, 0, 2] and b_next.item() == 4
    with pytest.raises(pkg.AbsError):
        ctx.abs_next_batch(stats, pkg.make_test_cfg("norm", 0, eta=0.5), b_cur, b_next, T_out)
    with pytest.raises(pkg.AbsError):
        ctx.abs_next_batch(stats, pkg.make_test_cfg("norm", 8, eta=0.0), b_cur, b_next, T_out)


# ------------------------------------------------------------------ full-size launch configuration
def _tiled_reference(small, d, b):
    """Statistics of the column-periodic extension of `small` [b, d0] to width d, assembled from
    oracle results on the block and on its first (d mod d0) columns: V, N and c_i are sums over
    columns, so K whole periods contribute K times the block's value."""
    d0 = small.shape[1]
    K, r = divmod(d, d0)
    A = orc.batch_test_stats(small)
    V = K * A["var_norm"]
    N = K * A["gbar_sq"]
    c = K * A["c"]
    if r:
        B = orc.batch_test_stats(small[:, :r])
        V += B["var_norm"]
        N += B["gbar_sq"]
        c = c + B["c"]
    var_ip = orc.batch_variance(c)
    return dict(gbar_sq=N, var_norm=V, var_ip=var_ip, var_orth=V - var_ip / N,
                sum_sq=(b - 1) * V + b * N, status=0, gbar=A["gbar"])


@pytest.mark.parametrize("b,d,offset,noise", [(64, 40000, 5.0, 0.01), (256, 9000, -300.0, 0.5), (1024, 3000, 2.0, 1e-3),
                                              (20, 50000, 1e3, 1.0)])
def test_mean_dominated_rows(ctx, b, d, offset, noise):
    """Rows that are a large common vector plus small noise: the centred accumulation keeps the
    variances at full accuracy although every entry is dominated by the mean."""
    gen = torch.Generator().manual_seed(b + d)
    common = offset * (1.0 + 0.1 * torch.randn(d, generator=gen))
    G = (common + noise * torch.randn((1, b, d), generator=gen)).cuda()
    recs, gbar = run_gpu(ctx, G)
    ref = orc.batch_test_stats(to_f64(G)[0])
    assert recs[0]["status"] == 0
    assert recs[0]["gbar_sq"] == pytest.approx(ref["gbar_sq"], rel=1e-5)
    assert recs[0]["var_norm"] == pytest.approx(ref["var_norm"], rel=1e-5)
    check_record(recs[0], ref, 1e-5, b)
    np.testing.assert_allclose(gbar[0].cpu().numpy(), ref["gbar"], rtol=1e-6)


@pytest.mark.parametrize("dtype,M,b,d,d0", [(torch.float32, 1, 256, 11_200_000, 100_003),
                                            (torch.float32, 1, 1024, 2_800_000, 50_003),
                                            (torch.bfloat16, 8, 16, 124_439_808, 250_007),
                                            (torch.bfloat16, 1, 64, 22_400_000, 100_003),
                                            (torch.bfloat16, 8, 128, 2_000_000, 100_003),
                                            (torch.bfloat16, 1, 256, 5_600_000, 50_003)])
def test_full_size_launch_configuration(ctx, dtype, M, b, d, d0):
    # the benchmark's launch shape (same b, M, dtype; d as large as a test should hold), checked
    # through the column-periodic property that holds at any width
    small = inputs.gaussian_rows(99, M, b, d0, 1.0, device="cuda").to(dtype)
    G = inputs.tile_columns(small, d)
    recs, gbar = run_gpu(ctx, G)
    H = to_f64(small)
    for m in range(M):
        ref = _tiled_reference(H[m], d, b)
        check_record(recs[m], ref, TOL[dtype], b)
        got = gbar[m, :d0].cpu().numpy()
        np.testing.assert_allclose(got, ref["gbar"], rtol=1e-5, atol=1e-6 * np.abs(ref["gbar"]).max())
        assert torch.equal(gbar[m, d0:2 * d0], gbar[m, :d0])


def _host_gib_free():
    with open("/proc/meminfo") as f:
        for line in f:
            if line.startswith("MemAvailable:"):
                return int(line.split()[1]) / (1 << 20)
    return 0.0


def _device_gib_free():
    torch.cuda.empty_cache()            # what earlier tests left in the caching allocator
    free, _ = torch.cuda.mem_get_info()
    return free / (1 << 30)


FULL_WIDTH = [
    # (dtype, b, d, recipe, route)   the oracle gets the whole matrix: every column is independent
    (torch.float32, 64, 11_200_000, "gauss", 2),       # tiled kernel, a column of the sweep
    (torch.float32, 64, 11_200_000, "gauss0.1", 2),    # the sweep's other noise levels: mean-dominated ...
    (torch.float32, 256, 2_800_000, "gauss10", 2),     # ... and noise-dominated
    (torch.float32, 16, 25_600_000, "gauss", 2),       # tiled kernel, widest rows of the sweep
    (torch.float32, 320, 2_800_000, "gauss", 1),       # cluster kernel (2 CTAs x 160 rows)
    (torch.float32, 1100, 1_000_000, "gauss", 1),      # cluster kernel, last CTA short of rows
    (torch.bfloat16, 16, 124_439_808, "student", 0),   # mma.sync Gram kernel at the LM width
    (torch.bfloat16, 64, 11_200_000, "gauss", 4),      # tcgen05 Gram kernel, one row block
    (torch.bfloat16, 160, 5_600_000, "gauss", 4),      # tcgen05 Gram kernel, two row blocks
]


@pytest.mark.parametrize("dtype,b,d,recipe,route", FULL_WIDTH)
def test_full_width_independent_columns_against_the_oracle(ctx, dtype, b, d, recipe, route):
    """Every statistics kernel against the oracle itself (not a periodic construction) on rows of
    10^6..10^8 independent columns: e_i = <g_i - gbar, gbar> is of order sigma ||gbar|| and is
    accumulated over all of them, in fp32 for 64 tiles / 4096 tensor-memory columns at a time before
    fp64 takes over.  No floor on var_ip: the tolerance is relative to var_ip itself."""
    need_host = b * d * 8 * 2.0 / (1 << 30)       # the fp64 copy and the widening's temporaries
    if _host_gib_free() < need_host + 4:
        pytest.skip("the oracle needs %.0f GiB of host memory for this case" % need_host)
    assert pkg.plan_stats("f32" if dtype == torch.float32 else "bf16", b)["route"] == route
    if recipe == "student":
        G = inputs.student_t_rows(31, 1, b, d, device="cuda", dtype=dtype)
    else:
        sigma = float(recipe[5:]) if len(recipe) > 5 else 1.0
        G = inputs.gaussian_rows(31 + b, 1, b, d, sigma, device="cuda", dtype=dtype)
    recs, gbar = run_gpu(ctx, G)
    H = to_f64(G)[0]
    del G
    ref = orc.batch_test_stats(H)
    check_record(recs[0], ref, TOL[dtype], b)
    assert recs[0]["recomputed"] == 0                     # noise-dominated rows: one pass over G
    np.testing.assert_allclose(gbar[0].cpu().numpy(), ref["gbar"], rtol=1e-5, atol=1e-6 * np.abs(ref["gbar"]).max())


def test_largest_sweep_cell_through_periodic_columns(ctx):
    """b = 1024, d = 25.6 M in fp32 (104.9 GB, one allocation): the cluster kernel's launch shape and
    64-bit indexing at the largest cell of the sweep, through the column-periodic property."""
    b, d, d0 = 1024, 25_600_000, 50_003
    if _device_gib_free() < b * d * 4 / (1 << 30) + 2:
        pytest.skip("the device cannot hold the 104.9 GB matrix")
    small = inputs.gaussian_rows(98, 1, b, d0, 1.0, device="cuda")
    G = inputs.tile_columns(small, d)
    recs, gbar = run_gpu(ctx, G)
    del G
    ref = _tiled_reference(to_f64(small)[0], d, b)
    check_record(recs[0], ref, 1e-5, b)
    np.testing.assert_allclose(gbar[0, :d0].cpu().numpy(), ref["gbar"], rtol=1e-5, atol=1e-6 * np.abs(ref["gbar"]).max())
    K = d // d0
    # the last whole period (it may come from the second launch, which adds the rows in another order)
    np.testing.assert_allclose(gbar[0, (K - 1) * d0:K * d0].cpu().numpy(), gbar[0, :d0].cpu().numpy(), rtol=1e-5,
                               atol=1e-6 * np.abs(ref["gbar"]).max())


@pytest.mark.parametrize("ratio", [10.0, 30.0, 100.0])
@pytest.mark.parametrize("b", [16, 64, 128, 256])
def test_mean_dominated_bf16_rows_through_the_gram_kernels(ctx, b, ratio):
    """bf16 rows that are a common vector `ratio` times the noise: the Gram kernels only ever see
    uncentred products added in fp32, so their variance is the difference of two sums of size
    sum_i ||g_i||^2 and loses b N / ((b-1) var_norm) in relative accuracy.  The finalisation measures
    that factor; beyond 25 (tcgen05 kernel) or 2500 (mma.sync kernel) the tiled kernel (centred
    accumulation) recomputes the record in a second pass.  Either way every statistic holds 1e-3;
    with the check switched off the Gram record of the worst cases does not."""
    d = 4_194_304
    gen = torch.Generator(device="cuda").manual_seed(1000 + b)
    common = ratio * (1.0 + 0.1 * torch.randn(d, device="cuda", generator=gen))
    G = torch.empty((1, b, d), device="cuda", dtype=torch.bfloat16)
    for i in range(b):
        G[0, i].copy_(common + torch.randn(d, device="cuda", generator=gen))
    assert pkg.plan_stats("bf16", b)["route"] == (0 if b <= 32 else 4)
    gram, gbar_g = run_gpu(ctx, G)
    ctx.set_tuning("stats_no_recheck", 1)
    try:
        unchecked, _ = run_gpu(ctx, G, want_gbar=False)
    finally:
        ctx.set_tuning("stats_no_recheck", 0)
    ctx.set_tuning("stats_no_gram", 1)
    try:
        tiled, _ = run_gpu(ctx, G, want_gbar=False)
    finally:
        ctx.set_tuning("stats_no_gram", 0)
    H = to_f64(G)[0]
    del G
    ref = orc.batch_test_stats(H)
    check_record(gram[0], ref, 1e-3, b)
    check_record(tiled[0], ref, 1e-3, b)
    np.testing.assert_allclose(gbar_g[0].cpu().numpy(), ref["gbar"], rtol=1e-5)
    kv = b * ref["gbar_sq"] / ((b - 1) * ref["var_norm"])          # about ratio^2
    limit = 2500.0 if b <= 32 else 25.0
    assert not 0.5 * limit < kv < 2.0 * limit                       # the cases are clear of the switch
    assert gram[0]["recomputed"] == (1 if kv > limit else 0)
    assert tiled[0]["recomputed"] == 0 and unchecked[0]["recomputed"] == 0
    if gram[0]["recomputed"]:
        for key in ("gbar_sq", "var_norm", "var_ip", "var_orth", "sum_sq"):
            assert gram[0][key] == tiled[0][key]                    # the same kernel produced both
    if b >= 64 and ratio >= 100.0:
        # what the check is for: the uncentred sums alone miss the tolerance here
        assert abs(unchecked[0]["var_norm"] - ref["var_norm"]) > 1e-3 * ref["var_norm"]


# ------------------------------------------------------------------ worker-gradient estimator (Section 4.3)
@pytest.mark.parametrize("M,b_local,d", [(4, 16, 30000), (8, 64, 12000), (2, 512, 5000)])
def test_worker_gradient_estimator(ctx, M, b_local, d):
    """The implemented test of the paper (Eq. test_stat_actual, Algorithm 2): the rows are the M workers'
    batch gradients, one row stands for b_local samples and the ratio carries an extra 1/M."""
    per_sample = inputs.gaussian_rows(123, M, b_local, d, 2.0, device="cuda")
    # the workers' batch gradients, produced by the library itself
    st = ctx.new_stats(M)
    Gb = torch.empty((M, d), device="cuda")
    ctx.abs_test_stats(per_sample, st, Gb)
    rows = Gb.unsqueeze(0)                                    # G[1, M, d]
    stats = ctx.new_stats(1)
    ctx.abs_test_stats(rows, stats)
    b_cur = torch.tensor([b_local], dtype=torch.int64, device="cuda")
    b_next = torch.zeros(1, dtype=torch.int64, device="cuda")
    T_out = torch.zeros(1, dtype=torch.int64, device="cuda")
    cfg = pkg.make_test_cfg("norm", 1 << 20, eta=0.5, row_weight=b_local, divisor=M)
    ctx.abs_next_batch(stats, cfg, b_cur, b_next, T_out)
    torch.cuda.synchronize()
    ref = orc.batch_test_stats(to_f64(Gb))
    rec = pkg.stats_to_dicts(stats)[0]
    check_record(rec, ref, 1e-5, M)
    exp_b, exp_T = orc.next_batch([rec], b_local, 1 << 20, "norm", eta=0.5, row_weight=b_local, divisor=M)
    assert T_out.tolist() == exp_T and b_next.item() == exp_b
    # Var_m(batch gradients) * b_local estimates the per-sample variance (2^2 * d here)
    if M >= 4:
        assert b_local * rec["var_norm"] == pytest.approx(4.0 * d, rel=0.1)


# ------------------------------------------------------------------ stream capture
@pytest.mark.parametrize("dtype,b", [(torch.float32, 256), (torch.float32, 1024), (torch.bfloat16, 16),
                                     (torch.bfloat16, 128)])
def test_a_step_can_be_captured_in_a_cuda_graph(ctx, dtype, b):
    """The calls only enqueue work (no allocation, no synchronisation), so a statistics + batch-size
    + optimiser step can be captured once and replayed: the replays give the eager results bit for bit."""
    M, d = 2, 20480
    G = make_G(55, M, b, d, dtype)
    cfg = pkg.make_test_cfg("aug_ip", 1 << 20, theta=0.5, nu=0.5)
    hp = dict(lr=1e-3, beta1=0.9, beta2=0.95, eps=1e-8, weight_decay=0.1)

    def fresh():
        X = torch.linspace(-1.0, 1.0, M * d, device="cuda").reshape(M, d).contiguous()
        return dict(X=X, m1=torch.zeros_like(X), m2=torch.zeros_like(X), gbar=torch.zeros((M, d), device="cuda"),
                    stats=ctx.new_stats(M), b_cur=torch.tensor([b], dtype=torch.int64, device="cuda"),
                    b_next=torch.zeros(1, dtype=torch.int64, device="cuda"))

    def step(st, t):
        ctx.abs_test_stats(G, st["stats"], st["gbar"])
        ctx.abs_next_batch(st["stats"], cfg, st["b_cur"], st["b_next"])
        ctx.local_adamw_step(st["X"], st["m1"], st["m2"], st["gbar"], pkg.make_adamw_cfg(step=t, **hp), average_after=1)

    eager = fresh()
    step(eager, 1)
    torch.cuda.synchronize()
    cap = fresh()
    graph = torch.cuda.CUDAGraph()
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step(cap, 1)                                   # warm-up outside the capture (function attributes)
        torch.cuda.synchronize()
        replay = fresh()
        with torch.cuda.graph(graph, stream=side):
            step(replay, 1)
    graph.replay()
    torch.cuda.synchronize()
    assert pkg.stats_to_dicts(replay["stats"]) == pkg.stats_to_dicts(eager["stats"])
    assert int(replay["b_next"].item()) == int(eager["b_next"].item())
    assert torch.equal(replay["X"], eager["X"]) and torch.equal(replay["m2"], eager["m2"])


# ------------------------------------------------------------------ bounded waits
@pytest.mark.parametrize("dtype,b", [(torch.float32, 40), (torch.bfloat16, 72), (torch.bfloat16, 200)])
def test_wait_that_runs_out_is_reported_and_the_context_stays_usable(ctx, dtype, b):
    """Failure detection without a fault: with the loader switched off no tile ever arrives, every
    wait gives up after its (shortened) limit, the kernel returns normally (the tcgen05 kernel
    frees its tensor memory) and the records carry ABS_STATUS_TIMEOUT; the next ordinary call on
    the same context is correct again.  Covers the tiled kernel and both shapes of the tcgen05 kernel."""
    G = make_G(77, 2, b, 6000, dtype)
    ctx.set_tuning("stats_no_cluster", 1)
    ctx.set_tuning("stats_timeout_cycles", 2_000_000)        # about a millisecond
    ctx.set_tuning("stats_fault_drop_loads", 1)
    try:
        flagged, _ = run_gpu(ctx, G, want_gbar=False)
    finally:
        ctx.set_tuning("stats_fault_drop_loads", 0)
        ctx.set_tuning("stats_timeout_cycles", 0)
        ctx.set_tuning("stats_no_cluster", 0)
    assert all(r["status"] & pkg.binding.STATUS_TIMEOUT for r in flagged)
    recs, _ = run_gpu(ctx, G, want_gbar=False)                # same context, ordinary call
    H = to_f64(G)
    for m in range(2):
        check_record(recs[m], orc.batch_test_stats(H[m]), TOL[dtype], b)


@pytest.mark.parametrize("dtype,b", [(torch.float32, 600), (torch.bfloat16, 1030)])
def test_cluster_kernel_wait_that_runs_out_is_reported(ctx, dtype, b):
    """The same for the cluster kernel (b > 256): no tile load is issued, the waits give up, nothing
    is left in flight, every CTA still reaches the cluster's last barrier and the launch ends."""
    assert pkg.plan_stats("f32" if dtype == torch.float32 else "bf16", b)["route"] == 1
    G = make_G(78, 2, b, 3000, dtype)
    ctx.set_tuning("stats_timeout_cycles", 2_000_000)
    ctx.set_tuning("stats_fault_drop_loads", 1)
    try:
        flagged, _ = run_gpu(ctx, G, want_gbar=False)
    finally:
        ctx.set_tuning("stats_fault_drop_loads", 0)
        ctx.set_tuning("stats_timeout_cycles", 0)
    assert all(r["status"] & pkg.binding.STATUS_TIMEOUT for r in flagged)
    recs, _ = run_gpu(ctx, G, want_gbar=False)
    H = to_f64(G)
    for m in range(2):
        check_record(recs[m], orc.batch_test_stats(H[m]), TOL[dtype], b)


# ------------------------------------------------------------------ per-worker sizes, merged sub-batches
def test_per_worker_batch_sizes_with_heterogeneous_constants(ctx):
    M, b, d = 5, 24, 9000
    G = make_G(300, M, b, d, torch.float32, sigma=0.7)
    stats = ctx.new_stats(M)
    ctx.abs_test_stats(G, stats)
    etas = [0.3, 0.5, 0.8, 0.95, 0.5]
    cur = [24, 24, 24, 5000, 10]
    eta_dev = torch.tensor(etas, dtype=torch.float64, device="cuda")
    b_cur = torch.tensor(cur, dtype=torch.int64, device="cuda")
    b_next = torch.zeros(M, dtype=torch.int64, device="cuda")
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    cfg = pkg.make_test_cfg("norm", 4096, eta=0.5)
    ctx.abs_next_batch_local(stats, cfg, b_cur, b_next, eta_m=eta_dev, T_out=T_out)
    torch.cuda.synchronize()
    recs = pkg.stats_to_dicts(stats)
    exp_b, exp_T = orc.next_batch_local(recs, cur, 4096, "norm", eta_per_worker=etas)
    assert T_out.tolist() == exp_T and b_next.tolist() == exp_b
    # no per-worker constants: cfg.eta for everybody, and the augmented test
    for kind, kw in (("norm", dict(eta=0.5)), ("aug_ip", dict(theta=0.5, nu=0.5))):
        ctx.abs_next_batch_local(stats, pkg.make_test_cfg(kind, 4096, **kw), b_cur, b_next, T_out=T_out)
        exp_b, exp_T = orc.next_batch_local(recs, cur, 4096, kind, **kw)
        assert T_out.tolist() == exp_T and b_next.tolist() == exp_b


@pytest.mark.parametrize("M,d,chunks", [(1, 5000, (16, 16)), (3, 12345, (8, 24, 5, 2)), (2, 70001, (64, 3, 33))])
def test_statistics_accumulated_over_micro_batches(ctx, M, d, chunks):
    """Gradient accumulation: the rows arrive in sub-batches, each goes through abs_test_stats and is
    folded into a running (mean, record) pair; the result equals the statistics of the whole batch."""
    b = sum(chunks)
    G = make_G(400 + b, M, b, d, torch.float32, sigma=1.3)
    run_mean = torch.empty((M, d), device="cuda")
    run_rec = ctx.new_stats(M)
    part_mean = torch.empty((M, d), device="cuda")
    part_rec = ctx.new_stats(M)
    lo = 0
    for k, n in enumerate(chunks):
        rows = G[:, lo:lo + n]
        lo += n
        if k == 0:
            ctx.abs_test_stats(rows, run_rec, run_mean)
        else:
            ctx.abs_test_stats(rows, part_rec, part_mean)
            ctx.abs_stats_merge(run_mean, part_mean, run_rec, part_rec)
    torch.cuda.synchronize()
    recs = pkg.stats_to_dicts(run_rec)
    H = to_f64(G)
    b_cur = torch.tensor([b], dtype=torch.int64, device="cuda")
    b_next = torch.zeros(1, dtype=torch.int64, device="cuda")
    T_out = torch.zeros(M, dtype=torch.int64, device="cuda")
    for m in range(M):
        ref = orc.batch_test_stats(H[m])
        assert recs[m]["rows"] == b and recs[m]["status"] == pkg.binding.STATUS_NORM_ONLY
        for key in ("gbar_sq", "var_norm", "sum_sq"):
            assert recs[m][key] == pytest.approx(ref[key], rel=1e-5)
        np.testing.assert_allclose(run_mean[m].cpu().numpy(), ref["gbar"], rtol=1e-5,
                                   atol=2e-6 * np.abs(ref["gbar"]).max())
    # the merged records drive the norm test; the augmented test declines them
    ctx.abs_next_batch(run_rec, pkg.make_test_cfg("norm", 1 << 20, eta=0.5), b_cur, b_next, T_out)
    exp_b, exp_T = orc.next_batch(recs, b, 1 << 20, "norm", eta=0.5)
    assert T_out.tolist() == exp_T and b_next.item() == exp_b
    ctx.abs_next_batch(run_rec, pkg.make_test_cfg("aug_ip", 1 << 20, theta=0.5, nu=0.5), b_cur, b_next, T_out)
    assert T_out.tolist() == [0] * M and b_next.item() == b

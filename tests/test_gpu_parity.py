"""GPU parity: the CUDA library against the CPU oracle, bit for bit, through the C ABI."""
import ctypes

import numpy as np
import pytest
import torch

import paper_2009_09271_b200 as sc
import workloads as wl
from oracle import sparsify_oracle as O
from parity_util import assert_bits_equal, run_step_both

pytestmark = pytest.mark.gpu

SCHEMES = [sc.SC_TOPK, sc.SC_RANDK, sc.SC_RANDBLOCK, sc.SC_RANDBLOCK_WRAP]
TILE = 4096


@pytest.fixture(scope="module")
def ctx():
    c = sc.Context(max_n=(1 << 22) + 64, max_W=8, max_segments=64)
    yield c
    c.close()


def rand(n, seed, scale=1e-3):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(n, generator=g) * scale


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("n", [1, 2, 3, 31, 32, 33, 1023, 1024, 1025, TILE - 1, TILE, TILE + 1,
                               2 * TILE - 3, 3 * TILE + 5, 100_003])
def test_single_worker_sizes(ctx, scheme, n):
    g = rand(n, n).view(1, n)
    e = rand(n, n + 1).view(1, n)
    for k in sorted({0, 1, (n + 99) // 100, n // 2, n - 1, n} & set(range(n + 1))):
        run_step_both(ctx, scheme, g, e, [(0, n, k)], [1234 + k])


@pytest.mark.parametrize("n", [4095, 4096, 4097, 36_864, 40_959, 40_960, 40_961, 50_000, 65_535])
def test_topk_segment_size_classes(ctx, n):
    """Short segments (one CTA, shared memory; two size classes) against the sizes just above them, which
    take the multi-pass radix select: k from 1 to n, with ties across the threshold."""
    W = 2
    g = torch.stack([rand(n, 300 + w) for w in range(W)])
    g[:, ::7] = g[:, 3:4]                                   # every seventh element equal: ties at many thresholds
    e = torch.stack([rand(n, 310 + w, scale=1e-4) for w in range(W)])
    e[:, ::7] = 0.0
    for k in (1, n // 100, n // 7 + 3, n // 2, n - 1, n):
        run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [0] * W)
        assert ctx.sc_topk_path_counts() == (W, 0, 0)


def test_topk_short_and_long_segments_in_one_table(ctx):
    """All four size classes side by side in one call (short x 2, multi-pass, one-pass), several steps."""
    sizes = [17, 4096, 1, 30_000, 45_000, 70_000, 2_000, 40_960, 131_072 + 5, 300]
    segs, off = [], 0
    for i, n_s in enumerate(sizes):
        off += i % 3                                        # gaps: elements outside every segment stay untouched
        segs.append((off, n_s, max(1, n_s // (3 + i))))
        off += n_s
    n, W = off + 2, 3
    res = torch.stack([rand(n, 400 + w, scale=1e-4) for w in range(W)])
    for t in range(3):
        g = torch.stack([rand(n, 410 + 10 * t + w) for w in range(W)])
        res = run_step_both(ctx, sc.SC_TOPK, g, res, segs, [t] * W, use=["step", "split", "host"][t])
        workers_last_call = 1 if t == 2 else W              # the host-buffer step compresses worker by worker
        assert ctx.sc_topk_path_counts() == (8 * workers_last_call, 2 * workers_last_call, 0)


def test_topk_massive_ties_and_special_values(ctx):
    n = 3 * TILE + 17
    g = torch.zeros(1, n)
    e = torch.zeros(1, n)
    pos = torch.randperm(n, generator=torch.Generator().manual_seed(0))
    g[0, pos[:200]] = 1.0          # 200 equal large values, the rest exact zeros
    g[0, pos[200:300]] = -1.0
    for k in (1, 150, 299, 300, 301, 2000, n - 1):
        run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [0])
    sp = rand(n, 5).view(1, n)
    sp[0, 5] = float("inf"); sp[0, 77] = float("-inf"); sp[0, 4096] = float("nan")
    sp[0, 9:20] = 0.0; sp[0, 30:40] = -0.0
    tiny = torch.from_numpy(np.array([1, 2, 0x80000001, 0x80000003], np.uint32).view(np.float32).copy())
    sp[0, 100:104] = tiny
    for k in (1, 2, 3, 50, n - 30, n - 5, n):
        run_step_both(ctx, sc.SC_TOPK, sp, e, [(0, n, k)], [0])
    # all values equal: the first k coordinates win
    eq = torch.full((1, n), 0.25)
    for k in (1, 100, TILE, TILE + 1, n):
        run_step_both(ctx, sc.SC_TOPK, eq, e, [(0, n, k)], [0])
    # small integers: thousands of ties at every level
    ints = torch.randint(-5, 6, (1, n), generator=torch.Generator().manual_seed(2)).float()
    for k in (10, 1000, 5000, n // 2):
        run_step_both(ctx, sc.SC_TOPK, ints, e, [(0, n, k)], [0])


@pytest.mark.parametrize("scheme", SCHEMES)
def test_segments_unaligned_multiworker(ctx, scheme):
    sizes = [5, 64, 1, 4099, 33, 8192, 7, 12289, 2, 1000]
    W = 5
    segs = wl.segment_table(sizes, 1, 10)
    n = sum(sizes)
    g = torch.stack([rand(n, 100 + w) for w in range(W)])
    e = torch.stack([rand(n, 200 + w) for w in range(W)])
    run_step_both(ctx, scheme, g, e, segs, [7] * W)                       # shared coordinates
    run_step_both(ctx, scheme, g, e, segs, [7, 8, 9, 10, 11])             # per-worker coordinates
    run_step_both(ctx, scheme, g, e, segs, [7] * W, use="split")
    # a table with gaps: elements outside every segment are left alone
    gap = [(3, 100, 10), (200, 4096, 41), (5000, 13, 13), (6000, 9000, 0)]
    run_step_both(ctx, scheme, g, e, gap, [3] * W)


@pytest.mark.parametrize("scheme", SCHEMES)
def test_row_length_not_multiple_of_four(ctx, scheme):
    W, n = 3, 2 * TILE + 1            # rows 1 and 2 start misaligned
    g = torch.stack([rand(n, 300 + w) for w in range(W)])
    e = torch.stack([rand(n, 400 + w) for w in range(W)])
    run_step_both(ctx, scheme, g, e, [(0, n, 97)], [1, 1, 1])
    run_step_both(ctx, scheme, g, e, [(1, 4000, 40), (4001, n - 4001, 400)], [1, 2, 3])


@pytest.mark.parametrize("scheme", SCHEMES)
def test_multistep_error_feedback_c1(ctx, scheme):
    """Workload 1 at full size: n = 2^20, W = 4, k = 10,486, three steps with the
    residual carried from step to step."""
    w1 = wl.workload("c1")
    segs = wl.flat_table(w1.n, 1, 100)
    assert segs[0].k == 10_486
    e = torch.zeros(w1.W, w1.n)
    for t in range(w1.steps):
        g = torch.stack([wl.generate(w1, w, t, "cpu") for w in range(w1.W)])
        e = run_step_both(ctx, scheme, g, e, segs, [wl.step_seed(w1.base_seed, t)] * w1.W)


@pytest.mark.parametrize("scheme", SCHEMES)
def test_telescoping_on_integer_gradients(ctx, scheme):
    n, k, W, T = 20_000, 200, 2, 12
    e = torch.zeros(W, n)
    total = torch.zeros(W, n, dtype=torch.float64)
    sent = torch.zeros(W, n, dtype=torch.float64)
    dev_ctx = ctx
    for t in range(T):
        g = torch.stack([wl.gen_small_integers(n, wl.make_generator(9, w, t, "cpu"), "cpu") for w in range(W)])
        total += g
        gd, ed = g.cuda(), e.cuda()
        vals = torch.empty(W, k, device="cuda"); idx = torch.empty(W, k, device="cuda", dtype=torch.int32)
        dev_ctx.sc_compress_batch(scheme, gd, ed, [(0, n, k)], [t, t + 100], vals, idx)
        assert dev_ctx.sc_sync_status() == 0
        for w in range(W):
            sent[w, idx[w].long().cpu()] += vals[w].double().cpu()
        e = ed.cpu()
    assert torch.equal(sent + e.double(), total)


def test_reduced_resnet_shapes(ctx):
    """Workloads 2 and 3 with every tensor shrunk 16x (same count of segments, same mix
    of tiny and large tensors), 3 steps each with error feedback."""
    for name, schemes in (("c2", [sc.SC_RANDBLOCK]), ("c3", SCHEMES)):
        w = wl.workload(name)
        sizes = [max(1, s // 16) for s in w.sizes][:64] if name == "c3" else [max(1, s // 16) for s in w.sizes]
        num, den = w.densities[0]
        segs = wl.segment_table(sizes, num, den)
        n = sum(sizes)
        W = 4
        for scheme in schemes:
            e = torch.zeros(W, n)
            for t in range(3):
                g = torch.stack([wl.generate(w, ww, t, "cpu", sizes=sizes) for ww in range(W)])
                e = run_step_both(ctx, scheme, g, e, segs, [wl.step_seed(w.base_seed, t)] * W)


def test_lstm_like_zero_rows(ctx):
    """Workload 4 structure: embedding tensors with 95 % exactly-zero rows, so that the
    top-k threshold is zero and most kept entries are ties."""
    sizes = [650 * 300, 20_000, 20_000, 650 * 300, 301, 50_000]
    w4 = wl.workload("c4")
    W = 3
    n = sum(sizes)
    for num, den in ((1, 1000), (1, 100), (1, 10)):
        for scheme in (sc.SC_TOPK, sc.SC_RANDBLOCK):
            for segs in (wl.segment_table(sizes, num, den), wl.flat_table(n, num, den)):
                e = torch.zeros(W, n)
                for t in range(2):
                    g = torch.stack([wl.generate(w4, ww, t, "cpu", sizes=sizes) for ww in range(W)])
                    e = run_step_both(ctx, scheme, g, e, segs, [wl.step_seed(3, t)] * W)


BIG = 1 << 20          # segments of at least this many elements take the sampled-bracket top-k path


@pytest.mark.parametrize("n", [BIG, BIG + 5, 3 * BIG + 4099])
def test_topk_large_segment_all_densities(ctx, n):
    g = rand(n, 11).view(1, n)
    e = rand(n, 12).view(1, n)
    for k in (0, 1, 7, n // 10000, n // 100, n // 10, n // 2, n - 1, n):
        run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [0])
        assert ctx.sc_topk_path_counts() == (0, 1, 0), k       # continuous values: the one-pass path serves it


def test_topk_sample_large_enough_for_the_cluster_bracket(ctx):
    """From 2^15 sample keys up the bracket kernel runs as a cluster of CTAs; the sample grows with the kept
    fraction, so a quarter or a half kept on a million elements takes that path (and one per cent does not)."""
    n = (1 << 20) + 13
    W = 3
    g = torch.stack([rand(n, 21 + w) for w in range(W)])
    e = torch.stack([rand(n, 31 + w, scale=1e-4) for w in range(W)])
    for k in (n // 100, n // 4, n // 2):
        run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [3] * W)
        assert ctx.sc_topk_path_counts() == (0, W, 0), k
    # both kinds of sample in one call: a large and a small segment side by side
    segs = [(0, 900_000, 300_000), (900_000, n - 900_000, 1000)]
    run_step_both(ctx, sc.SC_TOPK, g, e, segs, [4] * W)
    assert ctx.sc_topk_path_counts() == (0, 2 * W, 0)


def test_row_of_more_than_8192_tiles():
    """Rows of 8192 tiles and more have their per-tile counts scanned by a cluster of CTAs."""
    n = 8200 * 4096 + 77
    own = sc.Context(max_n=n, max_W=1, max_segments=2)
    gen = torch.Generator().manual_seed(5)
    g = (torch.randn(n, generator=gen) * 1e-3).view(1, n)
    e = torch.zeros(1, n)
    for scheme in (sc.SC_TOPK, sc.SC_RANDK):
        run_step_both(own, scheme, g, e, [(0, n, n // 1000)], [8])
    run_step_both(own, sc.SC_RANDK, g, e, [(0, 20_000_003, 20_000), (20_000_003, n - 20_000_003, 5)], [9])
    own.close()


def test_topk_large_segment_misaligned_rows_and_mixed_table(ctx):
    W, n = 3, BIG + 4099                       # odd row length: rows 1, 2 start misaligned
    g = torch.stack([rand(n, 900 + w) for w in range(W)])
    e = torch.stack([rand(n, 950 + w) for w in range(W)])
    run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, n // 100)], [0] * W)
    # a table that mixes tiny, medium and large tensors, unaligned starts
    sizes = [7, BIG + 1, 64, 5000, BIG + BIG // 2 + 3, 33]
    segs = wl.segment_table(sizes, 1, 100)
    n2 = sum(sizes)
    g2 = torch.stack([rand(n2, 960 + w) * (1 + w) for w in range(2)])
    e2 = torch.stack([rand(n2, 970 + w) for w in range(2)])
    e2 = run_step_both(ctx, sc.SC_TOPK, g2, e2, segs, [0, 0])
    assert ctx.sc_topk_path_counts() == (8, 4, 0)
    run_step_both(ctx, sc.SC_TOPK, g2, e2, segs, [0, 0], use="host")


def test_topk_large_segment_massive_ties_in_one_pass(ctx):
    """Inputs whose threshold sits on one massive key value (all equal, mostly zero, few distinct values):
    the sample shows that value, its elements are counted per tile instead of listed, and the lowest
    coordinates among them are admitted; no second pass over the segment."""
    n = BIG + 77
    e = torch.zeros(1, n)
    eq = torch.full((1, n), -0.5)
    for k in (1, n // 100, n - 3, n):
        run_step_both(ctx, sc.SC_TOPK, eq, e, [(0, n, k)], [0])
        assert ctx.sc_topk_path_counts() == (0, 1, 0)
        d = ctx.sc_topk_path_detail()
        assert d["tie_key_seen"] == 1 and d["ties_admitted"] == 1, (k, d)
    z = torch.zeros(1, n)
    nz = torch.randperm(n, generator=torch.Generator().manual_seed(1))[: n // 20]
    z[0, nz] = rand(n // 20, 13)
    for k in (n // 100, n // 20 - 1, n // 20, n // 20 + 1, n // 10, n // 2):
        run_step_both(ctx, sc.SC_TOPK, z, e, [(0, n, k)], [0])
        assert ctx.sc_topk_path_counts() == (0, 1, 0), k
        d = ctx.sc_topk_path_detail()
        assert d["ties_admitted"] == (1 if k > n // 20 else 0), (k, d)
    # zeros of both signs and a residual that cancels part of the gradient exactly
    zz = z.clone()
    zz[0, ::3] = -zz[0, ::3]
    ee = torch.zeros(1, n)
    ee[0, nz[: n // 40]] = -zz[0, nz[: n // 40]]                    # p becomes +0 or -0 there
    for k in (n // 50, n // 30, n // 5):
        run_step_both(ctx, sc.SC_TOPK, zz, ee, [(0, n, k)], [0])
        assert ctx.sc_topk_path_counts() == (0, 1, 0), k
    ints = torch.randint(-3, 4, (1, n), generator=torch.Generator().manual_seed(2)).float()
    for k in (10, n // 100, n // 3):
        run_step_both(ctx, sc.SC_TOPK, ints, e, [(0, n, k)], [0])
    heavy = wl.gen_student_t(n, torch.Generator().manual_seed(3), "cpu").view(1, n)
    heavy[0, 17] = float("inf"); heavy[0, 4242] = float("nan")
    for k in (1, 2, 3, n // 1000):
        run_step_both(ctx, sc.SC_TOPK, heavy, e, [(0, n, k)], [0])


def test_topk_ties_multiworker_segments_and_steps(ctx):
    """Tie admission with several workers, several large segments (one of them starting misaligned), short
    segments in between and the residual carried over three steps (zeros turn into earlier leftovers)."""
    W = 3
    sizes = [BIG + 5, 300, 2 * BIG + 4099, 70_000, 5000]
    segs = wl.segment_table(sizes, 1, 8)
    n = sum(sizes)
    res = torch.zeros(W, n)
    for t in range(3):
        g = torch.zeros(W, n)
        for w in range(W):
            gen = torch.Generator().manual_seed(100 * t + w)
            rows = torch.rand(n // 64 + 1, generator=gen) < 0.06      # runs of 64 non-zero coordinates, the rest exact zeros
            mask = rows.repeat_interleave(64)[:n]
            g[w] = torch.randn(n, generator=gen) * 1e-3 * mask
        res = run_step_both(ctx, sc.SC_TOPK, g, res, segs, [t] * W, use=["step", "split", "step"][t])
        assert ctx.sc_topk_path_counts()[2] == 0


def test_topk_large_segment_two_massive_values_fall_back(ctx):
    """A threshold that falls between two massive key values cannot be isolated by the sample (the upper one
    would have to be listed as candidates and does not fit): the radix select serves the segment, and the
    result must not depend on that."""
    n = BIG + 77
    e = torch.zeros(1, n)
    v = torch.ones(1, n)
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(7))
    c3 = n * 3 // 10
    v[0, perm[:c3]] = -3.0
    v[0, perm[c3:2 * c3]] = 2.0
    for k in (c3 - 5, c3, c3 + 5):
        run_step_both(ctx, sc.SC_TOPK, v, e, [(0, n, k)], [0])
        assert ctx.sc_topk_path_counts() == (0, 0, 1), k
        assert ctx.sc_topk_path_detail()["failed_list_overflow"] + ctx.sc_topk_path_detail()["failed_bracket"] == 1
    # several workers, only one of which fails; a failed and a fine segment side by side
    W = 3
    g = torch.stack([v[0], rand(n, 31), rand(n, 32)])
    run_step_both(ctx, sc.SC_TOPK, g, torch.zeros(W, n), [(0, n, c3 + 5)], [0] * W)
    assert ctx.sc_topk_path_counts() == (0, 2, 1)
    half = n // 2
    run_step_both(ctx, sc.SC_TOPK, g, torch.zeros(W, n), [(0, half, half * 3 // 10), (half, n - half, 1000)], [0] * W)
    assert ctx.sc_topk_path_counts()[0] == 0


def test_topk_crowded_tiles_continue_in_the_pool(ctx):
    """All large values in one stretch of the segment: the tiles there hold far more bracket elements than
    their share of the list, and continue in the pool behind the regions (no fall-back)."""
    n = 3 * BIG + 123
    W = 2
    g = torch.stack([rand(n, 41 + w, scale=1e-6) for w in range(W)])
    g[:, BIG:BIG + BIG // 2] = torch.stack([rand(BIG // 2, 51 + w, scale=1.0) for w in range(W)])
    e = torch.zeros(W, n)
    for k in (n // 100, n // 10, BIG // 2 - 1000):
        run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [0] * W)
        assert ctx.sc_topk_path_counts() == (0, W, 0), k
    # the same with one region per tile (a segment of few tiles) inside a table of several segments
    segs = [(0, 2 * BIG, BIG // 3), (2 * BIG, n - 2 * BIG, 1000)]
    run_step_both(ctx, sc.SC_TOPK, g, e, segs, [0] * W)
    assert ctx.sc_topk_path_counts() == (0, 2 * W, 0)


def test_bounded_waits_run_out_and_the_context_stays_usable(ctx):
    """The fall-back kernel's two waits (grid barrier, look-back of the pack phase), run where what they wait
    for never arrives: each gives up after the limit, the status word reports the time-out once, and the next
    call is bit-exact again."""
    n = BIG + 77
    g, e = rand(n, 61).view(1, n), torch.zeros(1, n)
    ctx.sc_debug_set_poll_limits(2000, 2000)
    try:
        for which in (0, 1):
            ctx.sc_debug_wait_probe(which)
            assert ctx.sc_sync_status() == -5
            assert sc.strerror(-5) == "bounded device wait timed out"
            assert ctx.sc_sync_status() == 0                              # reported once, then cleared
            run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, n // 100)], [0])
    finally:
        ctx.sc_debug_set_poll_limits(0, 0)
    # with the default limits the fall-back itself (barriers and look-backs that do complete) is bit-exact
    v = torch.ones(1, n)
    v[0, : n // 3] = 2.0
    run_step_both(ctx, sc.SC_TOPK, v, e, [(0, n, n // 3 + 5)], [0])


def test_aggregate_generic_shared_and_collisions(ctx):
    rng = np.random.default_rng(0)
    W, n, k = 7, 50_001, 5000
    idx = np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    vals = (rng.standard_normal((W, k)) * 10.0 ** rng.uniform(-3, 3, (W, k))).astype(np.float32)
    vals[0, :10] = -0.0
    d_idx = torch.from_numpy(idx.view(np.int32)).cuda()
    d_vals = torch.from_numpy(vals).cuda()
    out = torch.full((n,), float("nan"), device="cuda")
    ctx.sc_aggregate(W, d_vals, d_idx, k, n, out)
    assert ctx.sc_sync_status() == 0
    assert_bits_equal(out, O.aggregate(list(vals), list(idx), n), "generic aggregate")
    out.fill_(float("nan"))
    ctx.sc_aggregate_shared(W, d_vals, d_idx[0].contiguous(), k, n, out)
    assert ctx.sc_sync_status() == 0
    assert_bits_equal(out, O.aggregate(list(vals), [idx[0]] * W, n), "shared aggregate")
    # k = 0: all zeros
    ctx.sc_aggregate(W, d_vals, d_idx, 0, n, out)
    assert ctx.sc_sync_status() == 0
    assert not out.any() and not (out.view(torch.int32) != 0).any()
    # every worker sends the same single coordinate, at the very end
    one_i = torch.full((W, 1), n - 1, dtype=torch.int32, device="cuda")
    one_v = torch.arange(1, W + 1, dtype=torch.float32, device="cuda").view(W, 1) * 0.1
    ctx.sc_aggregate(W, one_v, one_i, 1, n, out)
    want = O.aggregate(list(one_v.cpu().numpy()), list(one_i.cpu().numpy().view(np.uint32)), n)
    assert_bits_equal(out, want, "single coordinate")


@pytest.mark.parametrize("W,n,density,clumped", [
    (16, 300_000, 0.02, False), (5, 300_001, 0.05, False), (16, 262_144, 0.10, False),
    (3, 200_003, 0.18, False), (8, 150_000, 0.30, False), (6, 250_000, 0.04, True), (16, 99_999, 0.10, True)])
def test_aggregate_private_coordinates_by_density(ctx, W, n, density, clumped):
    """Private coordinate sets from 2 % to 30 % kept (each range of slice lengths has its own kernel);
    'clumped' puts most of every message into a few stretches of 1024 coordinates."""
    if W > 8:
        own = sc.Context(max_n=n, max_W=W, max_segments=1)
    else:
        own = ctx
    rng = np.random.default_rng(int(n + 1000 * density) + W)
    k = int(n * density)
    rows = []
    for w in range(W):
        if clumped:
            hot = rng.choice(n // 1024, 3, replace=False) * 1024
            pool = np.concatenate([np.arange(h, min(h + 1024, n)) for h in hot])
            take_hot = min(k * 3 // 4, pool.size - 7)
            a = rng.choice(pool, take_hot, replace=False)
            rest = np.setdiff1d(np.arange(n), a, assume_unique=False)
            b = rng.choice(rest, k - take_hot, replace=False)
            rows.append(np.sort(np.concatenate([a, b])))
        else:
            rows.append(np.sort(rng.choice(n, k, replace=False)))
    idx = np.stack(rows).astype(np.uint32)
    vals = (rng.standard_normal((W, k)) * 10.0 ** rng.uniform(-3, 3, (W, k))).astype(np.float32)
    out = torch.full((n,), float("nan"), device="cuda")
    own.sc_aggregate(W, torch.from_numpy(vals).cuda(), torch.from_numpy(idx.view(np.int32)).cuda(), k, n, out)
    assert own.sc_sync_status() == 0
    assert_bits_equal(out, O.aggregate(list(vals), list(idx), n), "aggregate by density")
    if own is not ctx:
        own.close()


@pytest.mark.parametrize("scheme", SCHEMES)
@pytest.mark.parametrize("gamma", [0.1, -2.5, 3.0e-4])
def test_step_size_is_one_fused_multiply_add(ctx, scheme, gamma):
    """p = gamma g + e with a single rounding (Algorithm 1, accumulate line), on small and large
    segments, over three steps so that the residual feeds back."""
    W, n = 3, (1 << 17) + 4099
    segs = [(0, 70_001, 701), (70_001, 5_000, 50), (75_001, n - 75_001, 4000)]
    res = torch.zeros(W, n)
    for t in range(3):
        g = torch.stack([rand(n, 1000 * t + w, scale=1.0) for w in range(W)])
        res = run_step_both(ctx, scheme, g, res, segs, [11 + t] * W, gamma=gamma)


def test_step_size_halfway_cases(ctx):
    """Inputs where rounding the product first would give another answer than the fused form."""
    a = np.float32(1.0) + np.float32(2.0 ** -23)
    n = 4096 + 64
    g = torch.full((1, n), float(a))
    e_vals = np.float32([2.0 ** -24, -(2.0 ** -24), 3 * 2.0 ** -24, 1.0, -1.0, 2.0 ** -47, 0.0, -0.0])
    e = torch.from_numpy(np.resize(e_vals, n).copy()).view(1, n)
    for scheme in SCHEMES:
        run_step_both(ctx, scheme, g, e, [(0, n, 64)], [5], gamma=float(a))


def test_wrap_block_that_wraps(ctx):
    """Seeds are searched (on the CPU) until the block of the large and of a small segment wraps."""
    W, n = 2, 200_000
    segs = [(0, 150_000, 60_000), (150_000, 50_000, 49_999)]
    seed = next(s for s in range(1000)
                if O.block_start_wrap(O.segment_seed(s, 0), 150_000) + 60_000 > 150_000
                and O.block_start_wrap(O.segment_seed(s, 1), 50_000) > 1)
    g = torch.stack([rand(n, 77 + w) for w in range(W)])
    res = torch.stack([rand(n, 99 + w, scale=1e-4) for w in range(W)])
    run_step_both(ctx, sc.SC_RANDBLOCK_WRAP, g, res, segs, [seed] * W)
    run_step_both(ctx, sc.SC_RANDBLOCK_WRAP, g, res, segs, [seed, seed + 1], use="split")


def test_host_buffer_step(ctx):
    W, n = 4, 3 * TILE + 9
    g = torch.stack([rand(n, 500 + w) for w in range(W)])
    e = torch.stack([rand(n, 600 + w) for w in range(W)])
    for scheme in SCHEMES:
        run_step_both(ctx, scheme, g, e, [(0, n, 123)], [5] * W, use="host")
        run_step_both(ctx, scheme, g, e, [(0, n, 123)], [5, 6, 7, 8], use="host")


def test_repeatable(ctx):
    """The same call twice gives the same bits (no dependence on scheduling)."""
    W, n, k = 4, 200_003, 2001
    g = torch.stack([rand(n, 700 + w) for w in range(W)]).cuda()
    e0 = torch.stack([rand(n, 800 + w) for w in range(W)]).cuda()
    res = []
    for _ in range(2):
        e = e0.clone()
        vals = torch.empty(W, k, device="cuda"); idx = torch.empty(W, k, device="cuda", dtype=torch.int32)
        out = torch.empty(n, device="cuda")
        ctx.sc_step(sc.SC_TOPK, g, e, [(0, n, k)], [0, 1, 2, 3], vals, idx, out)
        assert ctx.sc_sync_status() == 0
        res.append((vals.clone(), idx.clone(), out.clone(), e.clone()))
    for a, b in zip(*res):
        assert torch.equal(a.view(torch.int32), b.view(torch.int32))


def test_argument_errors_leave_buffers_untouched(ctx):
    n, k = 1000, 10
    g = rand(n, 1).cuda(); e = rand(n, 2).cuda(); e0 = e.clone()
    vals = torch.zeros(k, device="cuda"); idx = torch.zeros(k, device="cuda", dtype=torch.int32)
    lib = sc.load_library()
    h = ctx._h
    assert lib.sc_compress(h, 7, g.data_ptr(), e.data_ptr(), n, k, 0, vals.data_ptr(), idx.data_ptr(), None) == -1
    assert lib.sc_compress(h, 0, g.data_ptr(), e.data_ptr(), n, n + 1, 0, vals.data_ptr(), idx.data_ptr(), None) == -2
    assert lib.sc_compress(h, 0, None, e.data_ptr(), n, k, 0, vals.data_ptr(), idx.data_ptr(), None) == -1
    assert lib.sc_compress(h, 0, g.data_ptr() + 4, e.data_ptr(), n - 1, k, 0, vals.data_ptr(), idx.data_ptr(), None) == -1
    assert lib.sc_compress(h, 0, g.data_ptr(), e.data_ptr(), (1 << 22) + 65, k, 0, vals.data_ptr(), idx.data_ptr(), None) == -2
    assert lib.sc_aggregate(h, 0, vals.data_ptr(), idx.data_ptr(), k, n, e.data_ptr(), None) == -2
    assert lib.sc_aggregate(h, 1, vals.data_ptr(), idx.data_ptr(), n + 1, n, e.data_ptr(), None) == -2
    torch.cuda.synchronize()
    assert torch.equal(e, e0) and not vals.any()
    with pytest.raises(sc.SparseCommError):
        ctx.sc_compress(9, g, e, k, 0, vals, idx)
    assert sc.strerror(-2) == "size out of range"


@pytest.mark.parametrize("W", [1, 4, 7, 16])
def test_aggregate_apply_matches_dense_update(W):
    """x <- x - average(messages), touched coordinates only, against the oracle's dense form."""
    rng = np.random.default_rng(40 + W)
    n, k = 300_007, 9000
    c = sc.Context(max_n=n, max_W=16, max_segments=1)
    idx = np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    vals = (rng.standard_normal((W, k)) * 10.0 ** rng.uniform(-3, 3, (W, k))).astype(np.float32)
    vals[0, :5] = [np.inf, -np.inf, 0.0, -0.0, 1e-42]
    x0 = (rng.standard_normal(n) * 0.1).astype(np.float32)
    x0[idx[0][2]] = -0.0
    d_idx, d_vals = torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(vals).cuda()
    x = torch.from_numpy(x0).cuda()
    c.sc_aggregate_apply(W, d_vals, d_idx, k, n, x)
    assert c.sc_sync_status() == 0
    assert_bits_equal(x, O.aggregate_apply(x0, list(vals), list(idx)), "apply")
    xs = torch.from_numpy(x0).cuda()
    c.sc_aggregate_apply(W, d_vals, d_idx[0].contiguous(), k, n, xs, shared=True)
    assert c.sc_sync_status() == 0
    assert_bits_equal(xs, O.aggregate_apply(x0, list(vals), [idx[0]] * W), "apply shared")
    c.close()


def test_rejected_table_does_not_poison_the_cached_layout():
    """A segment table that fails validation after another one was accepted must leave the context able to
    serve the earlier table again (the cached layout is dropped, not half-updated)."""
    n = (1 << 20) + 4099
    own = sc.Context(max_n=n, max_W=2, max_segments=4)
    g = torch.stack([rand(n, 1200 + w) for w in range(2)])
    e = torch.stack([rand(n, 1210 + w, scale=1e-4) for w in range(2)])
    good = [(0, n, n // 100)]
    e1 = run_step_both(own, sc.SC_TOPK, g, e, good, [0, 0])
    lib, h = sc.load_library(), own._h
    gd, ed = g.cuda(), e1.cuda()
    ed0 = ed.clone()
    vals = torch.zeros(2, n // 2, device="cuda"); idx = torch.zeros(2, n // 2, device="cuda", dtype=torch.int32)
    seeds = (ctypes.c_uint64 * 2)(0, 0)
    # overlapping segments; a table whose dense lists want the other build of the streaming pass, then fails
    for bad in ([(0, n // 2 + 10, 5), (n // 2, n - n // 2, 5)],
                [(0, n // 2, n // 4), (n // 2 - 1, n // 2, 7)]):
        arr = (sc.binding.ScSegment * len(bad))(*[sc.binding.ScSegment(*b) for b in bad])
        rc = lib.sc_compress_batch(h, sc.SC_TOPK, 2, gd.data_ptr(), ed.data_ptr(), n, arr, len(bad), seeds,
                                   vals.data_ptr(), idx.data_ptr(), None)
        assert rc == -1
        torch.cuda.synchronize()
        assert torch.equal(ed, ed0) and not vals.any()
        run_step_both(own, sc.SC_TOPK, g, e1, good, [0, 0])              # the earlier table still gives the oracle's bits
        assert own.sc_topk_path_counts() == (0, 2, 0)
    own.close()


@pytest.mark.parametrize("W", [2, 4, 3])
def test_aggregate_apply_denormal_sums(W):
    """Sums and model values in the denormal range: average-then-subtract is two roundings, which a fused
    multiply-add would merge into one."""
    rng = np.random.default_rng(90 + W)
    n, k = 20_000, 3000
    c = sc.Context(max_n=n, max_W=4, max_segments=1)
    idx = np.stack([np.sort(rng.choice(n, k, replace=False)) for _ in range(W)]).astype(np.uint32)
    vals = rng.integers(1, 1 << 12, (W, k)).astype(np.uint32)            # denormals: tiny odd multiples of 2^-149
    vals |= rng.integers(0, 2, (W, k)).astype(np.uint32) << 31
    vals = vals.view(np.float32)
    x0 = rng.integers(1, 1 << 14, n).astype(np.uint32)
    x0 |= rng.integers(0, 2, n).astype(np.uint32) << 31
    x0 = x0.view(np.float32)
    d_idx, d_vals = torch.from_numpy(idx.view(np.int32)).cuda(), torch.from_numpy(vals.copy()).cuda()
    x = torch.from_numpy(x0.copy()).cuda()
    c.sc_aggregate_apply(W, d_vals, d_idx, k, n, x)
    assert c.sc_sync_status() == 0
    assert_bits_equal(x, O.aggregate_apply(x0, list(vals), list(idx)), "apply, denormals")
    xs = torch.from_numpy(x0.copy()).cuda()
    c.sc_aggregate_apply(W, d_vals, d_idx[0].contiguous(), k, n, xs, shared=True)
    assert c.sc_sync_status() == 0
    assert_bits_equal(xs, O.aggregate_apply(x0, list(vals), [idx[0]] * W), "apply shared, denormals")
    c.close()


@pytest.mark.parametrize("scheme", SCHEMES)
def test_step_apply_matches_step_then_update(ctx, scheme):
    """sc_step_apply: compress, then x <- x - average at the sent coordinates; the same bits as the dense form."""
    W, sizes = 4, [70_001, 300, 4099, 131_072 + 9]
    segs = [(s.offset, s.n, s.k) for s in wl.segment_table(sizes, 1, 50)]
    n, K = sum(sizes), sum(s[2] for s in segs)
    x0 = rand(n, 1500, scale=1.0)
    for seeds in ([3] * W, [3, 4, 5, 6]):
        g = torch.stack([rand(n, 1510 + w) for w in range(W)])
        e0 = torch.stack([rand(n, 1520 + w, scale=1e-4) for w in range(W)])
        e = e0.cuda().clone()
        x = x0.cuda().clone()
        vals = torch.empty(W, K, device="cuda"); idx = torch.empty(W, K, device="cuda", dtype=torch.int32)
        ctx.sc_step_apply(scheme, g.cuda(), e, segs, seeds, vals, idx, x)
        assert ctx.sc_sync_status() == 0
        ov, oi, oe, _ = O.step(scheme, [g[w].numpy() for w in range(W)], [e0[w].numpy() for w in range(W)], segs, seeds)
        for w in range(W):
            assert_bits_equal(e[w], oe[w], f"residual[w={w}]")
            assert_bits_equal(idx[w], oi[w], f"idx[w={w}]")
        assert_bits_equal(x, O.aggregate_apply(x0.numpy(), ov, oi), "model")


def test_user_stream_short_and_long_segments_side_by_side(ctx):
    """On a stream of the caller's, with short segments (served on a stream of the library's own, forked from
    and joined to the caller's) next to long ones: the result is complete when the caller's stream is."""
    sizes = [3000, BIG + 9, 50_000, 200, 131_072, 17]
    segs = [(s.offset, s.n, s.k) for s in wl.segment_table(sizes, 1, 64)]
    n, K, W = sum(sizes), sum(s[2] for s in segs), 3
    g = torch.stack([rand(n, 1700 + w) for w in range(W)])
    e0 = torch.stack([rand(n, 1710 + w, scale=1e-4) for w in range(W)])
    ov, oi, oe, oout = O.step(sc.SC_TOPK, [g[w].numpy() for w in range(W)], [e0[w].numpy() for w in range(W)], segs, [0] * W)
    stream = torch.cuda.Stream()
    gd = g.cuda()
    for _ in range(3):                                                   # back to back: scratch reuse across calls in stream order
        e = e0.cuda().clone()
        vals = torch.full((W, K), float("nan"), device="cuda"); idx = torch.full((W, K), -1, device="cuda", dtype=torch.int32)
        out = torch.full((n,), float("nan"), device="cuda")
        torch.cuda.synchronize()
        with torch.cuda.stream(stream):
            ctx.sc_step(sc.SC_TOPK, gd, e, segs, [0] * W, vals, idx, out, stream=stream)
            ctx.sc_step(sc.SC_TOPK, gd, e.clone(), segs, [0] * W, vals.clone(), idx.clone(), out.clone(), stream=stream)
        stream.synchronize()
        for w in range(W):
            assert_bits_equal(idx[w], oi[w], f"idx[w={w}]")
            assert_bits_equal(vals[w], ov[w], f"vals[w={w}]")
            assert_bits_equal(e[w], oe[w], f"residual[w={w}]")
        assert_bits_equal(out, oout, "aggregate")
    assert ctx.sc_sync_status(stream) == 0


def _sample_keys(n, k):
    """Sample size the library takes for a large segment (the same arithmetic as its host code; if that changes,
    the test below still passes but no longer constructs the periodic case it is meant for)."""
    q = k / n
    balance = 1048576.0 * ((n / 350e6) * (max(q, 1e-9) / 0.1) ** 0.5) ** (2.0 / 3.0)
    capacity = 230400.0 * q * (1.0 - q)
    m = int(max(balance, capacity))
    m = min(m, n // 16, 1 << 20)
    return max(m, 4096) & ~7


def test_topk_values_periodic_in_the_sampling_stride(ctx):
    """Large entries exactly one sampling stride apart (a hot column of a row-major matrix): an evenly spaced
    sample would hold nothing but large entries, or none.  The sample's sectors sit at hashed places inside their
    stretches, so the bracket holds and the segment is served in one pass."""
    found = None
    for n in range(1 << 21, (1 << 22) + 1, 8):
        k = n // 64
        S = _sample_keys(n, k) // 8
        if (n // 8) % S == 0 and (n // 8) // S >= 4:
            found = (n, k, (n // 8) // S)
            break
    assert found is not None
    n, k, stride = found
    g = rand(n, 1800, scale=1e-3).view(1, n)
    big = rand(n // 8 // stride * 8, 1801, scale=10.0)
    g.view(-1, 8)[::stride] = big.view(-1, 8)                           # every stride-th sector is large
    e = torch.zeros(1, n)
    run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [0])
    assert ctx.sc_topk_path_counts() == (0, 1, 0)
    g2 = g.roll(8 * (stride // 2), dims=1)                              # the same pattern, half a stride on
    run_step_both(ctx, sc.SC_TOPK, g2, e, [(0, n, k)], [0])
    assert ctx.sc_topk_path_counts() == (0, 1, 0)


def test_step_of_one_aligned_segment_takes_its_aggregate_bounds_from_the_topk_offsets(ctx):
    """A table of one large segment that covers rows on the 128-byte grid: sc_step hands the top-k step's
    per-tile message offsets to the aggregate instead of searching the messages; a worker whose segment was
    redone by the fall-back is searched as usual.  Sparse and dense messages (both tile sizes of the aggregate)."""
    n, W = BIG + 64, 3
    v = torch.ones(n)
    perm = torch.randperm(n, generator=torch.Generator().manual_seed(9))
    c3 = n * 3 // 10
    v[perm[:c3]] = -3.0
    v[perm[c3:2 * c3]] = 2.0
    g = torch.stack([rand(n, 1900), v, rand(n, 1901, scale=1.0)])
    e = torch.zeros(W, n)
    for k in (c3 + 5, n // 1000, 1, 0, n // 2):
        run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, k)], [0] * W)
    run_step_both(ctx, sc.SC_TOPK, g, e, [(0, n, c3 + 5)], [0] * W)
    assert ctx.sc_topk_path_counts() == (0, 2, 1)

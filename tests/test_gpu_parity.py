"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle
on the same seeded inputs.  Scores within 2e-3 relative / 1e-5 absolute; index
sets, rank rows, statistic integers and compacted rows exact (index sets up to
the tolerance band around the k-th score)."""
import numpy as np
import pytest
import torch

from oracle import asl_oracle as O
from paper_2601_07667_b200 import inputs as I

from asl_check import StatReplay, bits_of, check_layer, make_path, to_dev, with_fp8_keys

pytestmark = pytest.mark.gpu


def run_stack(wl, seed, layers=None):
    """Every layer of the stack through check_layer (scores, index sets, compaction and the
    stage-isolated statistic are asserted there).  The end-to-end decision (selection layer,
    argmin layer) is a discontinuous function of the scores: ranks of near-tied tokens may
    differ between fp32 and fp64 scores.  It is compared whenever the oracle's relative
    variance keeps a margin of ten times the GPU/oracle deviation from the threshold (and
    from the runner-up for the argmin); a case without that margin is ill-posed and only its
    deviation is returned."""
    path = make_path(wl)
    replay = StatReplay(wl)
    rels_gpu, rels_ref = [], []
    for layer in (range(wl.layers) if layers is None else layers):
        x = I.layer_inputs(wl, layer, seed)
        res = check_layer(path, wl, x, layer)
        recs = replay.step(path, layer, res)
        iso, e2e = recs[0]
        if iso["evaluated"] and iso["m"] > 0:
            rels_gpu.append(iso["rel"])
            rels_ref.append(e2e["rel"])
    decided = True
    if rels_gpu:
        g, r = np.array(rels_gpu), np.array(rels_ref)
        dev = float(np.abs(g - r).max())
        decided = float(np.abs(r - wl.tau).min()) >= 10 * dev
        if decided:
            for b in range(wl.batch):
                assert replay.on_gpu_scores[b].selected_layer == replay.on_ref_scores[b].selected_layer
        rs = np.sort(r)
        if len(rs) < 2 or rs[1] - rs[0] >= 10 * dev:
            assert int(np.argmin(g)) == int(np.argmin(r))
    path.close()
    return rels_gpu, rels_ref, decided


def test_c1_tiny_stack():
    _, _, decided = run_stack(I.workload("C1"), seed=0)
    assert decided, "the tiny stack must keep its margin from the threshold"


def test_c1_other_seed_planted_keys_are_kept():
    wl = I.workload("C1")
    path = make_path(wl)
    x = I.layer_inputs(wl, 0, seed=7)
    check_layer(path, wl, x, 0)
    idx = path.idx.cpu().numpy()
    for h, pos in enumerate(I.planted_positions(wl, 7)[0]):
        assert np.isin(pos, idx[h]).all()
    path.close()


@pytest.mark.parametrize("seqlens,budgets,w,S", [
    ((33,), (32,), 32, 7),            # one past token, k = 0: window only
    ((200,), (500,), 32, 7),          # budget >= n: keep everything
    ((129,), (40,), 32, 1),           # S = 1, one key past a tile edge
    ((1000, 257, 4097), (100, 257, 300), 16, 5),   # ragged batch, tile-edge lengths
    ((700,), (96,), 24, 3),           # window that is not a power of two
])
def test_edge_shapes(seqlens, budgets, w, S):
    wl = I.workload("C1", seqlens=seqlens, budgets=budgets, window=w, pool_kernel=S, layers=3, l_min=1, l_obs=2)
    run_stack(wl, seed=3)


@pytest.mark.parametrize("seqlens,w,S", [
    ((152, 156, 2032 + 32, 36), 32, 9),      # segments of 120, 124, 2032 and 4 past tokens (a warp pools 120): widest window of the kernel
    ((152, 156, 2032 + 32, 36), 32, 1),      # no neighbours at all
    ((1000 + 24, 484 + 24), 24, 3),          # one partial row per kv head (the CUDA-core scorer's layout)
    ((3000 + 64, 1200 + 64), 64, 11),        # a window beyond the kernel's reach: the general kernel on the same layout
    ((3000 + 64, 1201 + 64), 64, 7),         # second segment off a 16-byte boundary: the general kernel
])
def test_average_pooling_on_aligned_segments(seqlens, w, S):
    """Batches whose segments all start and end on 16-byte boundaries of the score rows take the pooling kernel
    without shared memory; lengths around a warp's 120 tokens, every window size it covers, and the neighbouring
    cases that fall back to the general kernel."""
    wl = I.workload("C1", seqlens=seqlens, budgets=tuple(w + max(1, (n - w) // 4) for n in seqlens), window=w, pool_kernel=S,
                    layers=2, l_min=1, l_obs=2)
    run_stack(wl, seed=6)


@pytest.mark.parametrize("Hq,Hk,w,mode,n", [
    (32, 8, 64, 0, 3000),     # 256-row chunks, average pooling (the 8B-shaped layout)
    (8, 2, 128, 0, 2500),     # two 256-row chunks per kv head, average pooling
    (8, 2, 32, 1, 2000),      # max pooling, two query heads per column half
    (16, 2, 64, 1, 2100),     # max pooling, two chunks per kv head
    (4, 2, 256, 1, 1500),     # window as large as a chunk
    (4, 4, 64, 0, 1111),      # no grouping: 64-row chunk
    (6, 2, 32, 0, 1000),      # 96-row chunk
    (28, 4, 64, 0, 2500),     # seven query heads per kv head: 448 rows in seven 64-row chunks
])
def test_scorer_shapes(Hq, Hk, w, mode, n):
    wl = I.workload("C3", n_q_heads=Hq, n_kv_heads=Hk, window=w, pool_mode=mode, seqlens=(n,), budgets=(w + 100,),
                    layers=2, l_min=1, l_obs=2)
    run_stack(wl, seed=5)


@pytest.mark.parametrize("ctas", [100, 37, 1])
def test_scorer_grid_sizes_that_do_not_divide_the_work(ctas):
    """Tiles, rows to fold and publish counts are dealt by CTA index modulo the grid: odd and tiny grids."""
    wl = I.workload("C3", seqlens=(128 * 45 + 17,), budgets=(300,), layers=2, l_min=1, l_obs=2)
    path = make_path(wl, score_ctas=ctas, tail_streams=2)
    for layer in range(2):
        check_layer(path, wl, I.layer_inputs(wl, layer, 4), layer)
    path.close()


def _strided_case(wl, seed):
    """K and V interleaved in one buffer (token stride 2*H_k*d, V behind K) and q_obs rows padded to 1.5 d."""
    Hq, Hk, d, w = wl.n_q_heads, wl.n_kv_heads, wl.head_dim, wl.window
    qs = (Hq * w * (d + d // 2) + 64, w * (d + d // 2), d + d // 2)
    ks = (2 * Hk * d, d)
    path = make_path(wl, q_stride=qs, k_stride=ks, v_stride=ks)
    for layer in range(2):
        x = I.layer_inputs(wl, layer, seed)
        n = x["k"].shape[0]
        kv = torch.full((n, 2, Hk, d), -3.0, dtype=torch.bfloat16, device="cuda")
        kv[:, 0] = to_dev(x["k"])
        kv[:, 1] = to_dev(x["v"])
        qbuf = torch.full((wl.batch * qs[0],), 7.0, dtype=torch.bfloat16, device="cuda")
        qv = torch.as_strided(qbuf, (wl.batch, Hq, w, d), qs + (1,))
        qv.copy_(to_dev(x["q_obs"]))
        check_layer(path, wl, x, layer, q_dev=qv, k_dev=kv[:, 0], v_dev=kv[:, 1])
    path.close()


def test_strided_inputs_on_the_tensor_core_scorer():
    _strided_case(I.workload("C3", seqlens=(2900,), budgets=(400,), layers=2, l_min=1, l_obs=2), 6)


def test_strided_inputs_on_the_cuda_core_scorer():
    _strided_case(I.workload("C1", seqlens=(1500, 700), budgets=(200, 100), window=24, layers=2, l_min=1, l_obs=2), 6)


@pytest.mark.parametrize("which,code", [(0, 91), (1, 92)])
def test_a_wait_that_cannot_end_surfaces_as_a_timeout_status(which, code):
    """The scorer's waits are bounded.  One warp waits 20 us on a barrier nobody arrives on / a counter
    nobody advances: the kernel returns by itself, the context reports ASL_ERR_TIMEOUT with the code of
    the wait, the report clears the error word, and the context keeps working."""
    from paper_2601_07667_b200 import binding as B
    wl = I.workload("C1", seqlens=(700,), budgets=(100,), layers=1)
    path = make_path(wl)
    assert B.asl_device_status(path.ctx) == (B.ASL_OK, 0)
    B.asl_selftest_bounded_wait(path.ctx, which, 20000)
    assert B.asl_device_status(path.ctx) == (B.ASL_ERR_TIMEOUT, code)
    assert B.asl_device_status(path.ctx) == (B.ASL_OK, 0)
    check_layer(path, wl, I.layer_inputs(wl, 0, 2), 0)                 # the context is still usable
    with pytest.raises(B.AslError):
        B.asl_selftest_bounded_wait(path.ctx, 2, 20000)
    with pytest.raises(B.AslError):
        B.asl_selftest_bounded_wait(path.ctx, 0, 10**9)                 # limits beyond 1 ms are refused
    path.close()


@pytest.mark.parametrize("Hq,Hk,w,mode,n", [
    (32, 8, 64, 0, 128 * 21 + 50),    # 256-row chunks, average pooling
    (8, 2, 32, 0, 3000),              # 128-row chunk
    (16, 2, 64, 1, 2100),             # max pooling, two chunks per kv head
    (28, 4, 64, 0, 1700),             # padded last chunk
])
def test_fp8_key_cache(Hq, Hk, w, mode, n):
    """K as FP8 (E4M3) codes with one scale per kv head: scores against the oracle on the dequantised
    keys (same tolerance), selection exact on the GPU's scores, K rows compacted as codes, V as bf16."""
    from paper_2601_07667_b200 import binding as B
    wl = I.workload("C3", n_q_heads=Hq, n_kv_heads=Hk, window=w, pool_mode=mode, seqlens=(n, n // 2 + 77),
                    budgets=(w + 200, w + 90), layers=2, l_min=1, l_obs=2)
    xs = [with_fp8_keys(I.layer_inputs(wl, l, 9)) for l in range(2)]
    d = wl.head_dim
    path = None
    for layer, x in enumerate(xs):
        if path is None or not np.array_equal(scale, x["k_scale"]):      # the scales belong to the plan
            if path is not None:
                path.close()
            scale = x["k_scale"]
            path = make_path(wl, k_dtype=B.ASL_K_FP8_E4M3, k_scale=[float(s) for s in scale])
        check_layer(path, wl, x, layer, check_stat=False)
        assert path.k_out.dtype == torch.uint8
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


def test_fp8_keys_are_refused_where_no_tensor_core_path_exists():
    from paper_2601_07667_b200 import binding as B
    ctx = B.asl_create(0)
    base = dict(n_q_heads=8, n_kv_heads=2, head_dim=128, window=24, pool_kernel=7, pool_mode=0,
                cu_seqlens=[0, 500], budgets=[64], l_min=1, l_obs=2, tau=0.3,
                q_stride=(8 * 24 * 128, 24 * 128, 128), k_stride=(256, 128), v_stride=(256, 128))
    with pytest.raises(B.AslError) as e:
        B.asl_plan(ctx, **base, k_dtype=B.ASL_K_FP8_E4M3, k_scale=[1.0, 1.0])       # W = 24: CUDA-core scorer only
    assert e.value.status == B.ASL_ERR_UNSUPPORTED
    ok = {**base, "window": 32, "q_stride": (8 * 32 * 128, 32 * 128, 128)}
    for bad in (dict(k_scale=None), dict(k_scale=[1.0, 0.0]), dict(k_scale=[1.0, float("inf")]), dict(k_stride=(264, 128))):
        with pytest.raises(B.AslError) as e:
            B.asl_plan(ctx, **{**ok, "k_dtype": B.ASL_K_FP8_E4M3, "k_scale": [1.0, 1.0], **bad})
        assert e.value.status == B.ASL_ERR_INVALID
    assert B.asl_plan(ctx, **ok, k_dtype=B.ASL_K_FP8_E4M3, k_scale=[0.5, 2.0]) > 0
    B.asl_destroy(ctx)


def test_logits_far_above_the_first_keys_of_a_row():
    """Keys whose logit exceeds the row's reference (the maximum over its first 32 keys) by more than
    fp32's exponent range, so that the plain pass-1 sums overflow: in the last 32 keys of a tile (redone
    from registers), in the middle of a tile (the tile is redone with running maxima), twice in a row."""
    from paper_2601_07667_b200 import binding as B
    from asl_check import assert_scores_close, oracle_layer
    Hq, Hk, w, n = 32, 8, 64, 3000
    wl = I.workload("C3", n_q_heads=Hq, n_kv_heads=Hk, window=w, seqlens=(n,), budgets=(w + 100,), layers=1, l_min=1,
                    l_obs=2)
    g = np.random.default_rng(12)
    q = np.ones((1, Hq, w, wl.head_dim), np.float32) * (1.0 + 0.25 * (np.arange(w) % 4))[None, None, :, None]
    k = g.normal(0.0, 0.25, size=(n, Hk, wl.head_dim)).astype(np.float32)
    # q.k / sqrt(d) = 11.3 a (.. 19.8 a for the largest rows): 100 .. 400 nats above the other keys
    for pos, a in ((100, 9.0), (128 * 7 + 40, 13.25), (128 * 7 + 41, 20.0), (128 * 15 + 127, 11.0), (128 * 16, 12.0)):
        k[pos] = a
    x = {"q_obs": I.f32_to_bf16_bits(q), "k": I.f32_to_bf16_bits(k)}
    path = make_path(wl)
    B.asl_score_layer(path.ctx, to_dev(x["q_obs"]), to_dev(x["k"]), path.scores_kv, path.scores_agg, path.workspace,
                      path.ws_bytes)
    torch.cuda.synchronize()
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    P_ref, agg_ref = oracle_layer(wl, x)
    kv = path.scores_kv.cpu().numpy()
    assert np.isfinite(kv).all()
    assert_scores_close(kv, P_ref, "scores_kv with overflowing logits")
    assert_scores_close(path.scores_agg.cpu().numpy(), agg_ref, "scores_agg with overflowing logits")
    assert P_ref[:, 128 * 7 + 41].min() > 1.0            # the largest key carries the rows' mass
    path.close()


def test_ragged_batch_small():
    wl = I.workload("C4", seqlens=(3000, 5001, 2177, 4096), budgets=(300, 500, 217, 409), layers=3)
    run_stack(wl, seed=1)


def test_max_pool_wide_gqa_small():
    wl = I.workload("C5", seqlens=(5000,), budgets=(600,), layers=4, l_min=1, l_obs=3)
    run_stack(wl, seed=2)


def test_topk_exact_ties_lowest_index_wins():
    """Quantised scores: the k-th boundary falls inside long runs of exact ties."""
    from paper_2601_07667_b200 import binding as B
    # odd lengths: the second request's segment and every head's row start off a 16-byte boundary
    wl = I.workload("C1", seqlens=(9001 + 32, 2503 + 32), budgets=(1500, 2503 + 32))
    path = make_path(wl)
    for levels in (3, 16, 200):
        s = I.quantised_scores(wl.n_kv_heads, path.sum_T, levels, seed=levels)
        path.scores_kv.copy_(torch.from_numpy(s))
        B.asl_select_topk(path.ctx, path.scores_kv, wl.n_kv_heads, path.idx, path.workspace, path.ws_bytes)
        torch.cuda.synchronize()
        idx = path.idx.cpu().numpy()
        for b in range(wl.batch):
            n, w = wl.seqlens[b], wl.window
            ts, ko, kept = int(path.t_off[b]), int(path.kept_off[b]), wl.kept(b)
            for h in range(wl.n_kv_heads):
                ref = O.select_topk(s[h, ts:ts + n - w].astype(np.float64), kept - w, n, w)
                assert (idx[h, ko:ko + kept] == ref).all()
    path.close()


def test_topk_long_segment_of_many_tiles():
    """A segment of 74 tiles: the k-th boundary and the runs of ties span tiles."""
    from paper_2601_07667_b200 import binding as B
    T, w = 300000, 32
    wl = I.workload("C1", seqlens=(T + w,), budgets=(5000,))
    path = make_path(wl)
    for levels in (5, 100000):
        s = I.quantised_scores(wl.n_kv_heads, T, levels, seed=levels)
        path.scores_kv.copy_(torch.from_numpy(s))
        B.asl_select_topk(path.ctx, path.scores_kv, wl.n_kv_heads, path.idx, path.workspace, path.ws_bytes)
        torch.cuda.synchronize()
        idx = path.idx.cpu().numpy()
        for h in range(wl.n_kv_heads):
            assert (idx[h] == O.select_topk(s[h].astype(np.float64), 5000 - w, T + w, w)).all()
    path.close()


def _topk_against_the_oracle(wl, scores):
    from paper_2601_07667_b200 import binding as B
    path = make_path(wl)
    assert scores.shape == (wl.n_kv_heads, path.sum_T)
    path.scores_kv.copy_(torch.from_numpy(scores))
    path.idx.fill_(-1)
    B.asl_select_topk(path.ctx, path.scores_kv, wl.n_kv_heads, path.idx, path.workspace, path.ws_bytes)
    torch.cuda.synchronize()
    idx = path.idx.cpu().numpy()
    for b in range(wl.batch):
        n, w = wl.seqlens[b], wl.window
        ts, ko, kept = int(path.t_off[b]), int(path.kept_off[b]), wl.kept(b)
        for h in range(wl.n_kv_heads):
            ref = O.select_topk(scores[h, ts:ts + n - w].astype(np.float64), kept - w, n, w)
            assert (idx[h, ko:ko + kept] == ref).all(), (b, h)
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


def test_topk_of_mid_sized_segments_heavy_tailed_scores():
    """Segments of 8 K to 256 K scores (one CTA per segment: a sampled bound, one pass, a short list): smooth
    heavy-tailed scores, rows that start off a 16-byte boundary, the shortest and the longest such segment."""
    w = 32
    for seqlens, budgets in (((131008 + w + 3, 40001 + w), (4096, 2000)), ((8192 + w,), (700,)), ((262144 + w,), (6000,))):
        wl = I.workload("C1", seqlens=seqlens, budgets=budgets)
        T = sum(n - w for n in seqlens)
        rng = np.random.default_rng(T)
        s = np.exp(rng.normal(-9.0, 1.5, size=(wl.n_kv_heads, T))).astype(np.float32)
        s[:, :4] += 0.5                      # a few sinks far above the rest
        _topk_against_the_oracle(wl, s)


def test_topk_of_mid_sized_segments_when_the_sampled_bound_fails():
    """The same kernel where its short list cannot be used: (i) three score levels, so that every score reaches
    any bound and the list overflows; (ii) the large scores sit exactly on the sampled positions, so that the
    sample overstates them and fewer than k scores reach the bound.  Either way the result is exact."""
    w = 32
    wl = I.workload("C1", seqlens=(50000 + w, 9000 + w), budgets=(3000, 500))
    _topk_against_the_oracle(wl, I.quantised_scores(wl.n_kv_heads, 59000, 3, seed=4))
    T = 16384
    wl = I.workload("C1", seqlens=(T + w,), budgets=(1000 + w,))
    rng = np.random.default_rng(5)
    s = rng.uniform(0.0, 1e-3, size=(wl.n_kv_heads, T)).astype(np.float32)
    sampled = (np.arange(4096, dtype=np.int64) * T) // 4096
    s[:, sampled[::13]] = rng.uniform(1.0, 2.0, size=(wl.n_kv_heads, sampled[::13].size)).astype(np.float32)
    _topk_against_the_oracle(wl, s)


def test_rank_rows_with_ties_and_statistic_on_planted_rank_rows():
    """asl_rank_stat alone: tied scores, and a ring whose statistic has a closed form."""
    from paper_2601_07667_b200 import binding as B
    T, w = 10000, 32
    wl = I.workload("C1", seqlens=(T + w,), budgets=(T + w,), l_min=0, l_obs=2)       # k = T
    path = make_path(wl)
    asc = torch.arange(T, dtype=torch.float32, device="cuda")
    for layer, agg in enumerate([asc, -asc]):                     # rank rows: reversed, identity
        path.scores_agg.copy_(agg)
        B.asl_rank_stat(path.ctx, path.scores_agg, layer, layer + 1, path.rank_ring, path.stat, path.workspace,
                        path.ws_bytes)
    torch.cuda.synchronize()
    st = path.read_stat()[0]
    assert st["evaluated"] == 1 and st["m"] == T and st["rows"] == 2
    assert st["var_top"] == pytest.approx((T * T - 1) / 12.0, rel=1e-14)       # reversed ranks, k = T
    assert st["rel"] == 1.0 and st["selected"] == 0
    ties = torch.from_numpy(I.quantised_scores(1, T, 7, seed=9)[0]).cuda()
    path.scores_agg.copy_(ties)
    B.asl_rank_stat(path.ctx, path.scores_agg, 2, 2, path.rank_ring, path.stat, path.workspace, path.ws_bytes)
    torch.cuda.synchronize()
    assert (path.rank_ring[0].cpu().numpy() == O.rank_desc(ties.cpu().numpy().astype(np.float64))).all()
    path.close()


def test_rank_row_of_a_long_segment():
    """More tiles than the scatter kernel scans by itself: the separate scan kernel runs."""
    from paper_2601_07667_b200 import binding as B
    T, w = 300001, 32
    wl = I.workload("C1", seqlens=(T + w,), budgets=(5000,), l_min=0, l_obs=2)
    path = make_path(wl)
    for layer, levels in enumerate((11, 1 << 20)):
        s = I.quantised_scores(1, T, levels, seed=levels)[0]
        s[::7] *= -1.0                                            # both signs
        path.scores_agg.copy_(torch.from_numpy(s))
        B.asl_rank_stat(path.ctx, path.scores_agg, layer, layer + 1, path.rank_ring, path.stat, path.workspace,
                        path.ws_bytes)
        torch.cuda.synchronize()
        assert (path.rank_ring[layer % 2].cpu().numpy() == O.rank_desc(s.astype(np.float64))).all()
    path.close()


def test_invalid_arguments_are_refused():
    from paper_2601_07667_b200 import binding as B
    ctx = B.asl_create(0)
    base = dict(n_q_heads=8, n_kv_heads=2, head_dim=128, window=32, pool_kernel=7, pool_mode=0,
                cu_seqlens=[0, 100], budgets=[64], l_min=1, l_obs=2, tau=0.3,
                q_stride=(8 * 32 * 128, 32 * 128, 128), k_stride=(256, 128), v_stride=(256, 128))
    assert B.asl_plan(ctx, **base) > 0
    for bad in (dict(pool_kernel=4), dict(cu_seqlens=[0, 32]), dict(budgets=[16]), dict(n_kv_heads=3),
                dict(l_obs=1), dict(k_stride=(256, 127)), dict(window=0)):
        with pytest.raises(B.AslError) as e:
            B.asl_plan(ctx, **{**base, **bad})
        assert e.value.status == B.ASL_ERR_INVALID
    B.asl_plan(ctx, **base)
    t = torch.zeros(1 << 20, dtype=torch.float32, device="cuda")
    with pytest.raises(B.AslError) as e:
        B.asl_score_layer(ctx, t, t, t, t, t, 16)
    assert e.value.status == B.ASL_ERR_WORKSPACE
    with pytest.raises(B.AslError) as e:
        B.asl_rank_stat(ctx, t, 0, 2, t, t, t, t.numel() * 4)            # n_rows > layer_idx + 1
    assert e.value.status == B.ASL_ERR_INVALID
    assert B.asl_device_status(ctx)[0] == B.ASL_OK
    B.asl_destroy(ctx)


def test_run_twice_is_bitwise_identical():
    wl = I.workload("C1")
    x = I.layer_inputs(wl, 1, seed=4)
    q, k, v = to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])
    outs = []
    for _ in range(2):
        path = make_path(wl)
        path.run_layer(q, k, v, 0)
        torch.cuda.synchronize()
        outs.append((path.scores_kv.clone(), path.scores_agg.clone(), path.idx.clone(), path.rank_ring.clone()))
        path.close()
    for a, b in zip(*outs):
        assert torch.equal(a, b)


def test_device_side_controller_latches_the_selection_and_gates_the_one_shot_topk():
    """ASL_CONTROLLER_LATCH: Algorithm 2's state machine runs on the device.  After the layer at
    which a request's statistic selects, its record and rank rows stay as they are, and
    asl_select_topk_gated writes the one-shot selection at exactly that layer.  Reference: the
    oracle's controller and select_tokens fed the GPU's own aggregate scores layer by layer."""
    import dataclasses
    from paper_2601_07667_b200 import binding as B
    # a per-token salience that grows with depth: the ranking settles, the relative variance falls
    base = I.workload("C4", seqlens=(3000, 5001, 2177), budgets=(300, 500, 217), layers=7, l_min=1, l_obs=3,
                      salience_start=0.0, salience_step=0.5)
    xs = [I.layer_inputs(base, l, seed=11) for l in range(base.layers)]
    dev = [(to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])) for x in xs]

    def run(wl, latch):
        path = make_path(wl)
        if latch:
            B.asl_set_controller(path.ctx, B.ASL_CONTROLLER_LATCH)
        sel = torch.full((1, path.sum_kept), -1, dtype=torch.int32, device="cuda")
        aggs, stats, rings = [], [], []
        for l in range(wl.layers):
            path.run_layer(*dev[l], l, overlap=False)
            B.asl_select_topk_gated(path.ctx, path.scores_agg, 1, sel, path.stat, l, path.workspace, path.ws_bytes)
            torch.cuda.synchronize()
            aggs.append(path.scores_agg.cpu().numpy().astype(np.float64))
            stats.append(path.read_stat().copy())
            rings.append(path.rank_ring.cpu().numpy().copy())
        assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
        out = (path, aggs, stats, rings, sel.cpu().numpy()[0])
        return out

    # without a threshold nothing selects: the relative variances of every layer, per request
    never = dataclasses.replace(base, tau=0.0)
    path0, aggs, stats0, _, sel0 = run(never, latch=False)
    assert (sel0 == -1).all()
    rel = np.array([[st[b]["rel"] for b in range(base.batch)] for st in stats0 if st[0]["evaluated"]])
    tau = float(min(np.median(rel[1:-1]), 0.999))                 # some requests select somewhere in the middle ...
    t_off, kept_off = path0.t_off, path0.kept_off
    path0.close()

    wl = dataclasses.replace(base, tau=tau)
    ctl = [O.SelectionController(wl.budgets[b], wl.window, wl.l_min, wl.l_obs, wl.tau) for b in range(wl.batch)]
    at_sel = {}
    for l in range(wl.layers):
        for b in range(wl.batch):
            T = wl.seqlens[b] - wl.window
            if ctl[b].selected_layer < 0:                        # one shot: the controller stops observing afterwards
                rec = ctl[b].step(l, aggs[l][t_off[b]:t_off[b] + T])
                if ctl[b].selected_layer == l:
                    at_sel[b] = rec
    sel_layers = [c.selected_layer for c in ctl]
    assert any(1 < s < wl.layers - 1 for s in sel_layers) and len(set(sel_layers)) > 1, (sel_layers, tau, rel)   # ... not all alike

    path, aggs1, stats, rings, sel = run(wl, latch=True)
    for l in range(wl.layers):
        assert np.array_equal(aggs1[l], aggs[l])                 # same inputs, same scores, bit for bit
    final = stats[-1]
    for b in range(wl.batch):
        T, kept = wl.seqlens[b] - wl.window, wl.kept(b)
        ts, ko = int(t_off[b]), int(kept_off[b])
        L = sel_layers[b]
        if L < 0:
            assert final[b]["selected"] == 0 and (sel[ko:ko + kept] == -1).all()
            continue
        ref = at_sel[b]
        assert final[b]["selected"] == 1 and final[b]["layer_idx"] == L
        assert int(final[b]["num"]) == ref["num"] and int(final[b]["m"]) == ref["m"] and int(final[b]["rows"]) == ref["rows"]
        assert abs(final[b]["rel"] - ref["rel"]) <= 1e-13 * abs(ref["rel"])
        for l in range(L, wl.layers):                            # record and rank rows frozen from the selection layer on
            assert stats[l][b] == stats[L][b]
            assert np.array_equal(rings[l][:, ts:ts + T], rings[L][:, ts:ts + T])
        want = O.select_tokens(aggs[L][ts:ts + T], wl.budgets[b], wl.seqlens[b], wl.window)
        assert np.array_equal(sel[ko:ko + kept], want)
    path.close()


def test_work_of_finished_requests_is_skipped_under_the_latch():
    """Algorithm 2 ends the method for a request at its selection layer.  With the device-side
    controller and the layer clock (LayerPath.set_controller) the scorer, the pooling, the per-head
    top-k and the compaction leave a finished request alone: the outputs of the requests still under
    observation are bit for bit those of the run that skips nothing, and everything a finished request
    owns (scores, kept lists, compacted cache, rank rows, record) stays as its selection layer left it."""
    import dataclasses
    from paper_2601_07667_b200 import binding as B
    base = I.workload("C4", seqlens=(3000, 5001, 2177), budgets=(300, 500, 217), layers=7, l_min=1, l_obs=3,
                      salience_start=0.0, salience_step=0.5)
    xs = [I.layer_inputs(base, l, seed=11) for l in range(base.layers)]
    dev = [(to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])) for x in xs]

    def run(wl, mode):
        """mode 0: report every layer; 1: latch, nothing skipped (no layer clock); 2: latch with skipping"""
        path = make_path(wl, tail_streams=2)
        if mode == 1:
            B.asl_set_controller(path.ctx, B.ASL_CONTROLLER_LATCH)
        elif mode == 2:
            path.set_controller(B.ASL_CONTROLLER_LATCH)
        snaps = []
        for l in range(wl.layers):
            path.run_layer(*dev[l], l)
            torch.cuda.synchronize()
            snaps.append({"kv": [t.cpu().numpy().copy() for t in path._kv], "agg": [t.cpu().numpy().copy() for t in path._agg],
                          "cur": path._cur, "idx": path.idx.cpu().numpy().copy(), "k": bits_of(path.k_out).copy(),
                          "v": bits_of(path.v_out).copy(), "ring": path.rank_ring.cpu().numpy().copy(),
                          "stat": path.read_stat().copy()})
        if mode == 2:
            # a new prompt on the same context: the requests that were left out are scored again (their
            # publish counters were advanced while they were skipped) and every layer comes out as before
            path.reset()
            for l in range(wl.layers):
                path.run_layer(*dev[l], l)
                torch.cuda.synchronize()
                assert np.array_equal(path.idx.cpu().numpy(), snaps[l]["idx"])
                assert np.array_equal(path.read_stat(), snaps[l]["stat"])
        assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
        launches = B.asl_launch_count(path.ctx)
        offs = (path.t_off, path.kept_off)
        path.close()
        return snaps, offs, launches

    never = dataclasses.replace(base, tau=0.0)
    s0, (t_off, kept_off), _ = run(never, 0)
    rel = np.array([[st["stat"][b]["rel"] for b in range(base.batch)] for st in s0 if st["stat"][0]["evaluated"]])
    wl = dataclasses.replace(base, tau=float(min(np.median(rel[1:-1]), 0.999)))
    full, _, _ = run(wl, 1)
    skip, _, _ = run(wl, 2)
    sel_layer = [int(full[-1]["stat"][b]["layer_idx"]) if full[-1]["stat"][b]["selected"] else -1 for b in range(wl.batch)]
    assert any(0 <= L < wl.layers - 2 for L in sel_layer), sel_layer          # somebody finishes with layers to go
    for l in range(wl.layers):
        for b in range(wl.batch):
            T, kept = wl.seqlens[b] - wl.window, wl.kept(b)
            ts, ko = int(t_off[b]), int(kept_off[b])
            L = sel_layer[b]
            seg = lambda sn: (sn["idx"][:, ko:ko + kept], sn["k"][:, ko:ko + kept], sn["v"][:, ko:ko + kept],
                              sn["ring"][:, ts:ts + T], sn["stat"][b])
            if L < 0 or l <= L:                                   # still observed at layer l: nothing may differ
                cur = skip[l]["cur"]
                assert cur == full[l]["cur"]
                assert np.array_equal(skip[l]["kv"][cur][:, ts:ts + T], full[l]["kv"][cur][:, ts:ts + T])
                assert np.array_equal(skip[l]["agg"][cur][ts:ts + T], full[l]["agg"][cur][ts:ts + T])
                for a_, b_ in zip(seg(skip[l]), seg(full[l])):
                    assert np.array_equal(a_, b_)
            else:                                                 # finished: as the selection layer left it
                for a_, b_ in zip(seg(skip[l]), seg(skip[L])):
                    assert np.array_equal(a_, b_)
                for i in range(2):
                    assert np.array_equal(skip[l]["kv"][i][:, ts:ts + T], skip[L]["kv"][i][:, ts:ts + T])
                    assert np.array_equal(skip[l]["agg"][i][ts:ts + T], skip[L]["agg"][i][ts:ts + T])


def test_layers_replayed_from_a_cuda_graph_match_the_calls():
    """LayerPath.capture: four layers (side streams included) recorded once and replayed three
    times give, each time, bit for bit what the same calls give; the scorer numbers its launches
    on the device, so a replay is not mistaken for the launch that was recorded."""
    from paper_2601_07667_b200 import binding as B
    wl = I.workload("C1", layers=4, l_min=1, l_obs=3)
    xs = [I.layer_inputs(wl, l, seed=6) for l in range(4)]
    dev = [(to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])) for x in xs]
    path = make_path(wl)
    def snapshot():
        torch.cuda.synchronize()
        return [t.clone() for t in (path.scores_kv, path.scores_agg, path.idx, path.k_out, path.v_out, path.rank_ring,
                                    path.stat)]
    for l in range(4):
        path.run_layer(*dev[l], l)
    path.join()
    want = snapshot()
    path.reset()
    graph = path.capture([(*dev[l], l) for l in range(4)])
    for _ in range(3):
        path.reset()
        graph.replay()
        got = snapshot()
        assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
        for a, b in zip(got, want):
            assert torch.equal(a, b)
    for l in range(4):                        # calls after a capture still work
        path.run_layer(*dev[l], l)
    path.join()
    torch.cuda.synchronize()
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


@pytest.mark.parametrize("Hq,Hk,w,mode,n", [(32, 8, 64, 0, 3000), (8, 2, 32, 1, 2000), (6, 2, 40, 0, 900),
                                            (28, 4, 64, 0, 1500), (6, 2, 32, 0, 700)])     # the last two: padded chunks
def test_one_pass_scoring_with_supplied_lse(Hq, Hk, w, mode, n):
    """asl_score_layer_lse fed the oracle's log-sum-exp gives the oracle's scores; asl_window_lse
    returns the denominators the two-pass call found (tensor-core shapes and the CUDA-core fallback)."""
    from paper_2601_07667_b200 import binding as B
    from asl_check import assert_scores_close, oracle_layer
    wl = I.workload("C3", n_q_heads=Hq, n_kv_heads=Hk, window=w, pool_mode=mode, seqlens=(n,), budgets=(w + 50,),
                    layers=1, l_min=1, l_obs=2)
    x = I.layer_inputs(wl, 0, seed=8)
    path = make_path(wl)
    q, k = to_dev(x["q_obs"]), to_dev(x["k"])
    lse_ref = O.window_lse(O.widen_bf16(x["q_obs"][0]), O.widen_bf16(x["k"]), wl.group)
    lse_dev = torch.from_numpy(lse_ref.astype(np.float32)).cuda().reshape(1, Hq, w)
    B.asl_score_layer_lse(path.ctx, q, k, lse_dev, path.scores_kv, path.scores_agg, path.workspace, path.ws_bytes)
    torch.cuda.synchronize()
    P_ref, agg_ref = oracle_layer(wl, x)
    assert_scores_close(path.scores_kv.cpu().numpy(), P_ref, "one-pass scores_kv")
    assert_scores_close(path.scores_agg.cpu().numpy(), agg_ref, "one-pass scores_agg")
    B.asl_score_layer(path.ctx, q, k, path.scores_kv, path.scores_agg, path.workspace, path.ws_bytes)
    got = torch.empty((1, Hq, w), dtype=torch.float32, device="cuda")
    B.asl_window_lse(path.ctx, path.workspace, path.ws_bytes, got)
    torch.cuda.synchronize()
    assert np.abs(got.cpu().numpy()[0].astype(np.float64) - lse_ref).max() <= 2e-4     # log domain, absolute
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


@pytest.mark.parametrize("Hq,Hk,w,mode,n", [(32, 8, 64, 0, 3000), (8, 2, 32, 1, 2000), (6, 2, 40, 0, 900)])
def test_scoring_in_two_halves_matches_the_single_call_and_the_oracle(Hq, Hk, w, mode, n):
    """asl_score_columns + asl_pool_scores on either workspace slot give the oracle's scores and,
    bit for bit, what asl_score_layer gives; the two slots do not disturb each other."""
    from paper_2601_07667_b200 import binding as B
    from asl_check import assert_scores_close, oracle_layer
    wl = I.workload("C3", n_q_heads=Hq, n_kv_heads=Hk, window=w, pool_mode=mode, seqlens=(n,), budgets=(w + 50,),
                    layers=2, l_min=1, l_obs=2)
    xs = [I.layer_inputs(wl, l, seed=21) for l in range(2)]
    path = make_path(wl)
    qs, ks = [to_dev(x["q_obs"]) for x in xs], [to_dev(x["k"]) for x in xs]
    whole = []
    for l in range(2):
        B.asl_score_layer(path.ctx, qs[l], ks[l], path.scores_kv, path.scores_agg, path.workspace, path.ws_bytes)
        whole.append((path.scores_kv.clone(), path.scores_agg.clone()))
    # both first halves before either second half: slot 1 must survive the run that fills slot 0
    B.asl_score_columns(path.ctx, qs[1], ks[1], None, path.workspace, path.ws_bytes, 1)
    B.asl_score_columns(path.ctx, qs[0], ks[0], None, path.workspace, path.ws_bytes, 0)
    for l in range(2):
        kv, agg = torch.empty_like(path.scores_kv), torch.empty_like(path.scores_agg)
        B.asl_pool_scores(path.ctx, path.workspace, path.ws_bytes, l, kv, agg)
        torch.cuda.synchronize()
        assert torch.equal(kv, whole[l][0]) and torch.equal(agg, whole[l][1])
        P_ref, agg_ref = oracle_layer(wl, xs[l])
        assert_scores_close(kv.cpu().numpy(), P_ref, "two-halves scores_kv")
        assert_scores_close(agg.cpu().numpy(), agg_ref, "two-halves scores_agg")
    with pytest.raises(B.AslError):
        B.asl_score_columns(path.ctx, qs[0], ks[0], None, path.workspace, path.ws_bytes, 2)
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


def test_one_shot_selection_and_hidden_state_gather():
    """Alg. 2 (one-shot selection): top-k of the aggregate (one head) plus window, then a row gather of a
    per-token tensor; ragged batch, rows of 200 bf16 values (400 bytes)."""
    from paper_2601_07667_b200 import binding as B
    wl = I.workload("C4", seqlens=(3000, 777, 4097), budgets=(300, 100, 5000), layers=1)
    path = make_path(wl)
    g = torch.Generator().manual_seed(5)
    agg = torch.rand(path.sum_T, generator=g).mul(50).round().div(50)          # ties
    hidden = torch.randn(wl.total_tokens, 200, generator=g).to(torch.bfloat16)
    path.scores_agg.copy_(agg)
    idx = torch.empty(path.sum_kept, dtype=torch.int32, device="cuda")
    out = torch.empty(path.sum_kept, 200, dtype=torch.bfloat16, device="cuda")
    hd = hidden.cuda()
    B.asl_select_topk(path.ctx, path.scores_agg, 1, idx, path.workspace, path.ws_bytes)
    B.asl_compact_rows(path.ctx, hd, idx, out, 400)
    torch.cuda.synchronize()
    idx_h, out_h = idx.cpu().numpy(), out.cpu()
    cu = wl.cu_seqlens()
    for b in range(wl.batch):
        n, w = wl.seqlens[b], wl.window
        ts, ko, kept = int(path.t_off[b]), int(path.kept_off[b]), wl.kept(b)
        ref = O.select_tokens(agg[ts:ts + n - w].numpy().astype(np.float64), wl.budgets[b], n, w)
        assert (idx_h[ko:ko + kept] == ref).all()
        assert torch.equal(out_h[ko:ko + kept], hidden[int(cu[b]) + torch.from_numpy(ref)])
    with pytest.raises(B.AslError):
        B.asl_compact_rows(path.ctx, hd, idx, out, 100)                          # not a multiple of 16
    path.close()

"""Shared helpers of the GPU parity tests: run the CUDA path through the C ABI
on a seeded workload and compare every output with the fp64 oracle."""
from __future__ import annotations

import numpy as np
import torch

from oracle import asl_oracle as O
from paper_2601_07667_b200 import inputs as I

SCORE_RTOL, SCORE_ATOL = 2e-3, 1e-5          # tolerance of the scores against the fp64 oracle


def make_path(wl, device=0, **launch):
    """LayerPath of a workload.  ``launch``: the launch configuration (``score_ctas``, ``tail_streams``) and
    non-default strides (``q_stride``, ``k_stride``, ``v_stride``); omitted = the library's defaults."""
    from paper_2601_07667_b200 import binding
    return binding.LayerPath(n_q_heads=wl.n_q_heads, n_kv_heads=wl.n_kv_heads, head_dim=wl.head_dim,
                             window=wl.window, pool_kernel=wl.pool_kernel, pool_mode=wl.pool_mode,
                             seqlens=wl.seqlens, budgets=wl.budgets, l_min=wl.l_min, l_obs=wl.l_obs, tau=wl.tau,
                             device=device, **launch)


def bench_launch(device=0, one_pass=False):
    """The launch configuration bench.py times by default: the persistent scorer on all but 16 SMs (all but
    32 for its one-pass step), the rest of the layer on two side streams."""
    import bench
    return bench.default_launch(torch.cuda.get_device_properties(device).multi_processor_count, one_pass)


def to_dev(bits: np.ndarray) -> torch.Tensor:
    """uint16 bf16 bit patterns -> bf16 tensor on cuda:0 (bit-preserving); uint8 FP8 codes -> uint8 tensor."""
    if bits.dtype == np.uint8:
        return torch.from_numpy(bits).cuda()
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


def bits_of(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.uint8:
        return t.cpu().numpy()
    return t.view(torch.int16).cpu().numpy().view(np.uint16)


def with_fp8_keys(x):
    """The layer's inputs with K replaced by its FP8 copy (codes + one scale per kv head)."""
    codes, scale = I.keys_to_fp8(x["k"])
    return {**x, "k": codes, "k_scale": scale}


def oracle_layer(wl, x):
    """Oracle P [H_k][sum_T] and agg [sum_T] (packed like the library's outputs)."""
    cu = wl.cu_seqlens()
    Ps, aggs = [], []
    for b in range(wl.batch):
        q = O.widen_bf16(x["q_obs"][b])
        if "k_scale" in x:                       # a quantised K cache: the keys are code x scale
            k = O.dequantised_keys(x["k"][cu[b]:cu[b + 1]], x["k_scale"])
        else:
            k = O.widen_bf16(x["k"][cu[b]:cu[b + 1]])
        P, agg = O.score_layer(q, k, wl.group, wl.pool_kernel, wl.pool_mode)
        Ps.append(P)
        aggs.append(agg)
    return np.concatenate(Ps, axis=1), np.concatenate(aggs)


def assert_scores_close(gpu: np.ndarray, ref: np.ndarray, what: str):
    err = np.abs(gpu.astype(np.float64) - ref)
    bound = SCORE_ATOL + SCORE_RTOL * np.abs(ref)
    bad = err > bound
    assert not bad.any(), (f"{what}: {int(bad.sum())} of {bad.size} outside tolerance; worst "
                           f"err {err.max():.3e} at {np.unravel_index(np.argmax(err / bound), err.shape)}")
    return float((err / bound).max())


def check_topk_against_oracle(idx_gpu: np.ndarray, ref_scores: np.ndarray, k: int, n: int, w: int, what: str):
    """Index list of one (request, head) against the fp64 scores: exact outside
    the tolerance band around the k-th oracle score, valid inside it."""
    T = n - w
    assert idx_gpu.shape[0] == k + w, what
    assert (np.diff(idx_gpu) > 0).all(), f"{what}: not strictly ascending"
    assert (idx_gpu[k:] == np.arange(T, n)).all(), f"{what}: window indices"
    kept = idx_gpu[:k]
    assert k == 0 or (kept.min() >= 0 and kept.max() < T), what
    if k == 0 or k == T:
        return 0
    s_sorted = np.sort(ref_scores)[::-1]
    s_k = s_sorted[k - 1]
    tol = SCORE_ATOL + SCORE_RTOL * abs(s_k)
    mask = np.zeros(T, dtype=bool)
    mask[kept] = True
    must = ref_scores > s_k + tol
    never = ref_scores < s_k - tol
    assert mask[must].all(), f"{what}: a token clearly above the boundary was dropped"
    assert not mask[never].any(), f"{what}: a token clearly below the boundary was kept"
    exact = O.select_topk(ref_scores, k, n, w)[:k]
    return int(k - np.isin(kept, exact).sum())       # how many fell in the band and differ


def check_layer(path, wl, x, layer_idx, *, q_dev=None, k_dev=None, v_dev=None, ref=None, check_stat=True):
    """Runs one layer on the GPU and checks a1..a5 against the oracle.  Returns
    a dict with the GPU's aggregate (fp64) and statistic record(s)."""
    q_dev = to_dev(x["q_obs"]) if q_dev is None else q_dev
    k_dev = to_dev(x["k"]) if k_dev is None else k_dev
    v_dev = to_dev(x["v"]) if v_dev is None else v_dev
    path.run_layer(q_dev, k_dev, v_dev, layer_idx)
    torch.cuda.synchronize()
    return verify_layer(path, wl, x, layer_idx, ref=ref, check_stat=check_stat)


def verify_layer(path, wl, x, layer_idx, *, ref=None, check_stat=True):
    """Checks what the path's buffers hold after layer ``layer_idx`` (however it was issued: call by
    call or replayed from a CUDA graph) against the oracle on the host inputs ``x``."""
    cu = wl.cu_seqlens()
    P_gpu = path.scores_kv.cpu().numpy()
    agg_gpu = path.scores_agg.cpu().numpy()
    idx_gpu = path.idx.cpu().numpy()
    P_ref, agg_ref = oracle_layer(wl, x) if ref is None else ref
    worst = assert_scores_close(P_gpu, P_ref, f"layer {layer_idx} scores_kv")
    assert_scores_close(agg_gpu, agg_ref, f"layer {layer_idx} scores_agg")
    band = 0
    kb, vb = bits_of(path.k_out), bits_of(path.v_out)
    for b in range(wl.batch):
        n, w = wl.seqlens[b], wl.window
        T, k = n - w, wl.kept(b) - w
        ts, ko = int(path.t_off[b]), int(path.kept_off[b])
        for h in range(wl.n_kv_heads):
            ids = idx_gpu[h, ko:ko + k + w].astype(np.int64)
            band += check_topk_against_oracle(ids, P_ref[h, ts:ts + T], k, n, w, f"layer {layer_idx} b{b} h{h}")
            # fed the GPU's own fp32 scores, the selection is exact (ties to the lower index)
            exact = O.select_topk(P_gpu[h, ts:ts + T].astype(np.float64), k, n, w)
            assert (ids == exact).all(), f"layer {layer_idx} b{b} h{h}: selection differs on identical scores"
            # compaction is a pure gather of the bf16 rows
            assert (kb[h, ko:ko + k + w] == O.compact_rows(x["k"][cu[b]:cu[b + 1]], ids, h)).all()
            assert (vb[h, ko:ko + k + w] == O.compact_rows(x["v"][cu[b]:cu[b + 1]], ids, h)).all()
    out = {"agg_gpu": agg_gpu.astype(np.float64), "agg_ref": agg_ref, "band": band, "worst": worst}
    if check_stat:
        out["stat"] = path.read_stat().copy()
        slot = layer_idx % wl.l_obs
        ring = path.rank_ring[slot].cpu().numpy()
        for b in range(wl.batch):
            ts, T = int(path.t_off[b]), wl.seqlens[b] - wl.window
            assert (ring[ts:ts + T] == O.rank_desc(out["agg_gpu"][ts:ts + T])).all(), \
                f"layer {layer_idx} b{b}: rank row differs from RankDesc of the same scores"
    return out


class StatReplay:
    """Oracle controllers fed the GPU's own aggregate scores (stage-isolated
    check of the rank statistic) and, separately, the oracle's scores."""

    def __init__(self, wl):
        mk = lambda b: O.SelectionController(wl.budgets[b], wl.window, wl.l_min, wl.l_obs, wl.tau)
        self.on_gpu_scores = [mk(b) for b in range(wl.batch)]
        self.on_ref_scores = [mk(b) for b in range(wl.batch)]
        self.wl = wl

    def step(self, path, layer_idx, res):
        wl = self.wl
        recs = []
        for b in range(wl.batch):
            ts, T = int(path.t_off[b]), wl.seqlens[b] - wl.window
            iso = self.on_gpu_scores[b].step(layer_idx, res["agg_gpu"][ts:ts + T])
            e2e = self.on_ref_scores[b].step(layer_idx, res["agg_ref"][ts:ts + T])
            s = res["stat"][b]
            assert int(s["evaluated"]) == int(iso["evaluated"]), f"layer {layer_idx} b{b}"
            if iso["evaluated"]:
                assert int(s["num"]) == iso["num"] and int(s["m"]) == iso["m"] and int(s["rows"]) == iso["rows"]
                if iso["m"] == 0:          # k = 0: empty union, the statistic is undefined and never selects
                    assert np.isnan(s["var_top"]) and np.isnan(s["rel"]) and np.isnan(iso["rel"])
                else:
                    assert abs(s["var_top"] - iso["var_top"]) <= 1e-14 * abs(iso["var_top"])
                    if np.isnan(iso["rel"]):   # the first evaluated layer had zero variance: the ratio is undefined and never selects
                        assert np.isnan(s["rel"]) and not bool(s["selected"])
                    else:
                        assert abs(s["rel"] - iso["rel"]) <= 1e-13 * abs(iso["rel"])
                assert bool(s["selected"]) == iso["selected"]
            recs.append((iso, e2e))
        return recs

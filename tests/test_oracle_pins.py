"""Pins for the fp64 oracle: closed forms, invariants, brute force and library
cross-checks.  None of them re-types the oracle's own formula; each is chosen
so that a plausible slip (wrong scale, mask off by one, transposed operand,
wrong GQA mapping, wrong divisor, unstable tie order) fails at least one."""
import itertools
import math
import statistics

import numpy as np
import pytest
import torch

from oracle import asl_oracle as O
from paper_2601_07667_b200 import inputs as I


def rng(seed):
    return np.random.default_rng(seed)


# ------------------------------------------------------------------ O1 / O2
def brute_force_U(q, k, group):
    """Pure-Python loops, log-sum-exp formulation, math.fsum accumulation."""
    Hq, w, d = q.shape
    n = k.shape[0]
    T = n - w
    U = [[0.0] * T for _ in range(Hq)]
    for a in range(Hq):
        h = a // group
        cols = [[] for _ in range(T)]
        for t in range(w):
            last = T + t
            logits = [math.fsum(float(q[a, t, c]) * float(k[j, h, c]) for c in range(d)) / math.sqrt(d)
                      for j in range(last + 1)]
            mx = max(logits)
            lse = mx + math.log(math.fsum(math.exp(x - mx) for x in logits))
            for j in range(T):
                cols[j].append(math.exp(logits[j] - lse))
        for j in range(T):
            U[a][j] = math.fsum(cols[j])
    return np.array(U)


@pytest.mark.parametrize("n,w,Hq,Hk,d", [(9, 1, 2, 1, 4), (24, 5, 4, 2, 8), (40, 8, 6, 2, 16), (33, 32, 2, 2, 4)])
def test_U_brute_force(n, w, Hq, Hk, d):
    g = rng(n * 7 + w)
    q = g.standard_normal((Hq, w, d)) * 2.0
    k = g.standard_normal((n, Hk, d)) * 2.0
    U = O.past_column_sums(q, k, Hq // Hk)
    assert np.allclose(U, brute_force_U(q, k, Hq // Hk), rtol=1e-12, atol=1e-15)


def test_rows_sum_to_one_and_total_mass_is_w():
    g = rng(1)
    Hq, Hk, w, d, n = 8, 2, 16, 32, 300
    q = g.standard_normal((Hq, w, d)); k = g.standard_normal((n, Hk, d))
    for a in range(Hq):
        A = O.window_attention(q[a], k[:, a // 4, :])
        assert (A >= 0).all()
        assert np.allclose(A.sum(axis=1), 1.0, atol=1e-13)
    U, wm = O.past_column_sums(q, k, 4, return_window_mass=True)
    assert np.allclose(U.sum(axis=1) + wm, w, atol=1e-11)     # all n columns total w per q head
    assert (U.sum(axis=1) <= w).all()


def test_causal_mask_on_last_block():
    g = rng(2)
    w, d, n = 6, 8, 20
    A = O.window_attention(g.standard_normal((w, d)), g.standard_normal((n, d)))
    T = n - w
    for t in range(w):
        assert (A[t, T + t + 1:] == 0).all()          # row t never sees keys after its own position
        assert A[t, T + t] > 0                        # ... but does see itself
        assert (A[t, :T] > 0).all()                   # and every past key


def test_identical_keys_closed_form():
    # all keys equal -> row t is uniform over its T+t+1 visible keys
    g = rng(3)
    Hq, w, d, n = 2, 7, 8, 50
    T = n - w
    q = g.standard_normal((Hq, w, d))
    k = np.tile(g.standard_normal((1, 1, d)), (n, 1, 1))
    U = O.past_column_sums(q, k, 2)
    expect = sum(1.0 / (T + t + 1) for t in range(w))
    assert np.allclose(U, expect, rtol=1e-13)
    # zero queries give the same
    U0 = O.past_column_sums(np.zeros((Hq, w, d)), g.standard_normal((n, 1, d)), 2)
    assert np.allclose(U0, expect, rtol=1e-13)


def test_scale_is_one_over_sqrt_d():
    # one key with logit c/sqrt(d), all others 0: p = e^x / (e^x + visible - 1)
    d, w, n = 4, 3, 10
    T = n - w
    c = 3.0
    q = np.zeros((1, w, d)); q[0, :, 0] = c
    k = np.zeros((n, 1, d)); k[2, 0, 0] = 1.0
    U = O.past_column_sums(q, k, 1)
    x = c / math.sqrt(d)
    expect2 = sum(math.exp(x) / (math.exp(x) + (T + t + 1) - 1) for t in range(w))
    expect_other = sum(1.0 / (math.exp(x) + (T + t + 1) - 1) for t in range(w))
    assert U[0, 2] == pytest.approx(expect2, rel=1e-13)
    assert np.allclose(np.delete(U[0], 2), expect_other, rtol=1e-13)


def test_dominant_key_takes_every_row():
    g = rng(4)
    Hq, w, d, n = 2, 5, 8, 30
    q = np.abs(g.standard_normal((Hq, w, d))) + 0.5
    k = g.standard_normal((n, 1, d)) * 0.01
    k[11, 0, :] = 200.0
    U = O.past_column_sums(q, k, 2)
    assert np.allclose(U[:, 11], w, atol=1e-9)
    assert np.delete(U, 11, axis=1).max() < 1e-9


def test_w1_is_textbook_softmax():
    g = rng(5)
    d, n = 16, 37
    q = g.standard_normal((1, 1, d)); k = g.standard_normal((n, 1, d))
    U = O.past_column_sums(q, k, 1)
    ref = torch.softmax(torch.from_numpy(k[:, 0, :] @ q[0, 0]) / math.sqrt(d), dim=0).numpy()
    assert np.allclose(U[0], ref[: n - 1], rtol=1e-12)


def test_gqa_head_mapping_contiguous_groups():
    g = rng(6)
    Hq, Hk, w, d, n = 6, 3, 4, 8, 25
    q = g.standard_normal((Hq, w, d)); k = g.standard_normal((n, Hk, d))
    U = O.past_column_sums(q, k, 2)
    k2 = k.copy(); k2[:, 1, :] = g.standard_normal((n, d))      # change kv head 1 only
    U2 = O.past_column_sums(q, k2, 2)
    changed = [not np.allclose(U[a], U2[a]) for a in range(Hq)]
    assert changed == [False, False, True, True, False, False]


def test_widen_bf16_exact():
    bits = np.array([0x3F80, 0xBF80, 0x4049, 0x0000, 0x3E00, 0x7F7F], dtype=np.uint16)
    ref = torch.from_numpy(bits.view(np.int16)).view(torch.bfloat16).to(torch.float64).numpy()
    assert (O.widen_bf16(bits) == ref).all()
    assert O.widen_bf16(bits)[2] == 3.140625


# ------------------------------------------------------------------ O3 / O4
@pytest.mark.parametrize("S", [1, 3, 5, 7, 9])
def test_pool_matches_library(S):
    g = rng(10 + S)
    U = g.random((3, 41))
    t = torch.from_numpy(U)[None]
    avg = torch.nn.functional.avg_pool1d(t, S, stride=1, padding=S // 2)[0].numpy()
    mx = torch.nn.functional.max_pool1d(t, S, stride=1, padding=S // 2)[0].numpy()
    assert np.allclose(O.pool1d(U, S, O.POOL_AVG), avg, rtol=1e-14, atol=0)
    assert (O.pool1d(U, S, O.POOL_MAX) == mx).all()


def test_pool_closed_forms():
    T, S = 20, 7
    r = S // 2
    assert (O.pool1d(rng(0).random((2, T)), 1) == rng(0).random((2, T))).all()      # S=1 identity
    delta = np.zeros((1, T)); delta[0, 9] = 1.0
    box = O.pool1d(delta, S)
    assert np.allclose(box[0, 9 - r: 9 + r + 1], 1.0 / S) and box.sum() == pytest.approx(1.0)
    assert (O.pool1d(delta, S, O.POOL_MAX)[0] == np.r_[np.zeros(6), np.ones(7), np.zeros(7)]).all()
    const = np.full((1, T), 2.5)
    out = O.pool1d(const, S)[0]
    assert np.allclose(out[r: T - r], 2.5)
    for i in range(r):                      # zero padding, fixed divisor
        assert out[i] == pytest.approx(2.5 * (r + 1 + i) / S)
        assert out[T - 1 - i] == pytest.approx(2.5 * (r + 1 + i) / S)
    with pytest.raises(ValueError):
        O.pool1d(const, 4)


def test_pool_then_group_sum_is_linear_for_avg():
    g = rng(11)
    U = g.random((8, 50))
    a = O.sum_groups(O.pool1d(U, 7), 4)
    b = O.pool1d(O.sum_groups(U, 4), 7)
    assert np.allclose(a, b, rtol=1e-13)
    assert O.sum_groups(np.arange(12.0).reshape(4, 3), 2).tolist() == [[3, 5, 7], [15, 17, 19]]
    assert O.aggregate_scores(np.arange(12.0).reshape(4, 3)).tolist() == [18, 22, 26]


# ------------------------------------------------------------------ O5
def test_rank_desc_brute_force_and_ties():
    g = rng(20)
    s = g.integers(0, 12, size=200).astype(np.float64)        # many ties
    r = O.rank_desc(s)
    assert sorted(r.tolist()) == list(range(200))
    for j in range(200):
        expect = int((s > s[j]).sum() + (s[:j] == s[j]).sum())
        assert r[j] == expect
    assert O.rank_desc(np.array([5.0, 4.0, 3.0, 2.0])).tolist() == [0, 1, 2, 3]
    assert O.rank_desc(np.array([1.0, 3.0, 3.0, 2.0])).tolist() == [3, 0, 1, 2]


# ------------------------------------------------------------------ O6
def test_rank_statistic_closed_forms():
    T = 101
    ident = np.arange(T)
    num, m, var = O.rank_statistic(np.stack([ident] * 4), 10)
    assert (num, m, var) == (0, 10, 0.0)
    num, m, var = O.rank_statistic(np.stack([ident, ident[::-1]]), T)
    assert m == T
    assert var == pytest.approx((T * T - 1) / 12.0, rel=1e-14)     # mean of ((T-1-2r)/2)^2
    # union semantics: k smallest ranks of EACH row
    R = np.array([[0, 1, 2, 3, 4], [4, 3, 2, 1, 0]])
    num, m, var = O.rank_statistic(R, 1)
    assert m == 2 and var == pytest.approx(4.0)                    # tokens 0 and 4: ranks {0,4}
    num, m, var = O.rank_statistic(R, 2)
    assert m == 4 and var == pytest.approx((4 + 1 + 1 + 4) / 4)


def test_rank_statistic_brute_force_sets():
    g = rng(30)
    for trial in range(20):
        T = int(g.integers(4, 33)); rows = int(g.integers(2, 6)); k = int(g.integers(1, T + 1))
        R = np.stack([g.permutation(T) for _ in range(rows)])
        union = set()
        for r in range(rows):
            union |= set(sorted(range(T), key=lambda j: R[r][j])[:k])
        expect = statistics.fmean(statistics.pvariance([int(R[r][j]) for r in range(rows)]) for j in sorted(union))
        num, m, var = O.rank_statistic(R, k)
        assert m == len(union) and k <= m <= min(T, k * rows)
        assert var == pytest.approx(expect, rel=1e-12)
        assert num == round(var * rows * rows * m)


def test_rank_statistic_random_permutations_mean():
    g = rng(31)
    T, rows = 200, 4
    vals = [O.rank_statistic(np.stack([g.permutation(T) for _ in range(rows)]), T)[2] for _ in range(200)]
    expect = (rows - 1) / rows * (T * T - 1) / 12.0
    assert np.mean(vals) == pytest.approx(expect, rel=0.02)


def test_controller_policy():
    g = rng(32)
    T = 300
    base = g.random(T)
    layers = 12
    # fresh noise fades with depth -> ranks stabilise -> relative variance falls
    aggs = [base + g.random(T) * (1.5 * (0.6 ** l)) for l in range(layers)]
    sel = []
    for tau in (0.05, 0.2, 0.4, 0.7, 1.0, 1.1):
        c = O.SelectionController(budget=64 + 8, window=8, l_min=3, l_obs=3, tau=tau)
        outs = [c.step(l, aggs[l]) for l in range(layers)]
        assert not any(o["evaluated"] for o in outs[:3])            # layer < L_min -> None
        first = next(o for o in outs if o["evaluated"])
        assert first["layer"] == 3 and first["rel"] == 1.0 and first["rows"] == 3
        assert all(o["rows"] == 3 for o in outs if o["evaluated"])
        sel.append(c.selected_layer if c.selected_layer >= 0 else layers)
    assert sel == sorted(sel, reverse=True)                          # L_sel non-increasing in tau
    assert sel[0] > sel[-1]
    assert sel[-1] == 3          # rel = 1 at the first evaluated layer: fires there only if tau > 1
    assert sel[-2] > 3           # the comparison is strict: rel = 1.0 is not < 1.0


def test_controller_after_a_first_layer_without_variance():
    """Rank rows that agree on the union at the first evaluated layer give var_top = 0: every later ratio to
    it is undefined (NaN) and the strict comparison never fires, whatever the threshold."""
    T = 40
    same = np.linspace(1.0, 0.0, T)                      # the same order at every layer: identical rank rows
    c = O.SelectionController(budget=8 + 4, window=4, l_min=1, l_obs=2, tau=10.0)
    outs = [c.step(l, same) for l in range(2)]
    assert outs[1]["evaluated"] and outs[1]["var_top"] == 0.0 and np.isnan(outs[1]["rel"]) and not outs[1]["selected"]
    moved = same.copy()
    moved[[0, 30]] = moved[[30, 0]]                      # now the rows differ: the variance is positive, the ratio still undefined
    out = c.step(2, moved)
    assert out["var_top"] > 0.0 and np.isnan(out["rel"]) and not out["selected"] and c.selected_layer < 0


# ------------------------------------------------------------------ O7 / O8
def test_select_topk_brute_force_ties_and_edges():
    g = rng(40)
    n, w = 70, 6
    T = n - w
    P = g.integers(0, 9, size=T).astype(np.float64)
    for k in (0, 1, 7, 30, T):
        idx = O.select_topk(P, k, n, w)
        assert idx.size == k + w and (np.diff(idx) > 0).all()
        assert idx[k:].tolist() == list(range(T, n))
        kept = set(idx[:k].tolist())
        expect = set(sorted(range(T), key=lambda j: (-P[j], j))[:k])
        assert kept == expect
        dropped = [P[j] for j in range(T) if j not in kept]
        if kept and dropped:
            assert min(P[j] for j in kept) >= max(dropped)
    assert O.select_topk(np.array([1.0, 1.0, 1.0, 1.0]), 2, 6, 2).tolist() == [0, 1, 4, 5]
    assert O.kept_count(512, 4096, 32) == 480 and O.kept_count(9999, 100, 32) == 68
    assert O.kept_count(2048, 32768, 64) == min(2048 - 64, 32768 - 64)     # both formulas for k agree


def test_compact_rows_is_a_gather():
    g = rng(41)
    x = g.integers(0, 65536, size=(20, 3, 8)).astype(np.uint16)
    idx = np.array([1, 4, 19])
    out = O.compact_rows(x, idx, 2)
    assert out.dtype == np.uint16 and (out == np.stack([x[1, 2], x[4, 2], x[19, 2]])).all()
    assert (O.compact_rows(x, np.arange(20), 0) == x[:, 0, :]).all()


def test_score_layer_composition_small():
    g = rng(42)
    Hq, Hk, w, d, n, S = 4, 2, 3, 8, 30, 5
    q = g.standard_normal((Hq, w, d)); k = g.standard_normal((n, Hk, d))
    P, agg = O.score_layer(q, k, 2, S)
    U = brute_force_U(q, k, 2)
    t = torch.from_numpy(U)[None]
    Vp = torch.nn.functional.avg_pool1d(t, S, stride=1, padding=S // 2)[0].numpy()
    assert np.allclose(P, Vp[0::2] + Vp[1::2], rtol=1e-12)
    assert np.allclose(agg, Vp.sum(axis=0), rtol=1e-12)
    Pm, _ = O.score_layer(q, k, 2, S, O.POOL_MAX)
    Vm = torch.nn.functional.max_pool1d(t, S, stride=1, padding=S // 2)[0].numpy()
    assert np.allclose(Pm, Vm[0::2] + Vm[1::2], rtol=1e-12)


# ------------------------------------------------------------------ window log-sum-exp
def test_window_lse_closed_form_and_brute_force():
    g = rng(21)
    Hq, Hk, w, d, n = 4, 2, 5, 8, 30
    T = n - w
    # identical keys: every visible logit equals s, so lse = s + log(number of visible keys)
    key = g.standard_normal(d)
    k = np.broadcast_to(key, (n, Hk, d)).copy()
    q = g.standard_normal((Hq, w, d))
    lse = O.window_lse(q, k, Hq // Hk)
    for a in range(Hq):
        for t in range(w):
            s = float(q[a, t] @ key) / math.sqrt(d)
            assert lse[a, t] == pytest.approx(s + math.log(T + t + 1), abs=1e-12)
    # random keys: pure-Python sums, and the defining property A = exp(s - lse)
    k = g.standard_normal((n, Hk, d)) * 2.0
    lse = O.window_lse(q, k, Hq // Hk)
    for a in range(Hq):
        A = O.window_attention(q[a], k[:, a // 2, :])
        for t in range(w):
            logits = [math.fsum(float(q[a, t, c]) * float(k[j, a // 2, c]) for c in range(d)) / math.sqrt(d)
                      for j in range(T + t + 1)]
            brute = math.log(math.fsum(math.exp(x) for x in logits))
            assert lse[a, t] == pytest.approx(brute, abs=1e-12)
            assert A[t, 3] == pytest.approx(math.exp(logits[3] - lse[a, t]), rel=1e-12)


def test_select_tokens_is_the_union_of_best_ranks_and_window():
    g = rng(33)
    T, w, budget = 50, 6, 16
    agg = g.integers(0, 8, size=T).astype(np.float64)          # many ties
    sel = O.select_tokens(agg, budget, T + w, w)
    k = budget - w
    assert sel.shape[0] == k + w and (np.diff(sel) > 0).all()
    assert (sel[k:] == np.arange(T, T + w)).all()
    order = sorted(range(T), key=lambda j: (-agg[j], j))        # brute force: best k, ties to the lower index
    assert sorted(order[:k]) == sel[:k].tolist()
    assert (O.select_tokens(agg, 10 ** 6, T + w, w) == np.arange(T + w)).all()      # budget >= n keeps everything


# ---------------------------------------------------------------- FP8 (E4M3) keys
def test_fp8_e4m3_decode_literal_values():
    """Bit patterns whose values follow from the format's definition: 1 sign, 4 exponent bits (bias 7),
    3 mantissa bits, subnormals at exponent 0, largest finite value 448, S.1111.111 is NaN."""
    codes = np.array([0x00, 0x80, 0x38, 0xB8, 0x40, 0x3C, 0x7E, 0xFE, 0x01, 0x07, 0x08, 0x30, 0x47], dtype=np.uint8)
    want = [0.0, -0.0, 1.0, -1.0, 2.0, 1.5, 448.0, -448.0, 2.0 ** -9, 7 * 2.0 ** -9, 2.0 ** -6, 0.5, 3.75]
    got = O.widen_fp8_e4m3(codes)
    assert got.tolist() == want
    assert np.signbit(got[1]) and not np.signbit(got[0])
    assert np.isnan(O.widen_fp8_e4m3(np.array([0x7F, 0xFF], dtype=np.uint8))).all()


def test_fp8_e4m3_decode_agrees_with_the_library_type_on_all_codes():
    codes = np.arange(256, dtype=np.uint8)
    lib = torch.from_numpy(codes.copy()).view(torch.float8_e4m3fn).to(torch.float64).numpy()
    got = O.widen_fp8_e4m3(codes)
    assert np.array_equal(np.isnan(got), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(got[ok], lib[ok]) and np.array_equal(np.signbit(got[ok]), np.signbit(lib[ok]))
    # strictly increasing over the positive codes, symmetric in the sign bit
    assert (np.diff(got[0:0x7F]) > 0).all() and np.array_equal(got[0x80:0xFF], -got[0x00:0x7F])


def test_fp8_key_copy_is_the_nearest_code_and_scales_per_head():
    """The input helper's codes: no other code is nearer to k/scale, the head's largest key maps to 448."""
    g = np.random.default_rng(5)
    k = (g.standard_normal((40, 3, 16)) * np.array([0.3, 1.0, 20.0])[None, :, None]).astype(np.float32)
    bits = I.f32_to_bf16_bits(k)
    codes, scale = I.keys_to_fp8(bits)
    assert codes.dtype == np.uint8 and codes.shape == k.shape and scale.shape == (3,)
    exact = I.bf16_bits_to_f64(bits) / scale.astype(np.float64)[None, :, None]
    table = O.widen_fp8_e4m3(np.arange(0x7F, dtype=np.uint8))             # all non-negative finite values
    err = np.abs(np.abs(O.widen_fp8_e4m3(codes)) - np.abs(exact))
    best = np.abs(np.abs(exact)[..., None] - table).min(axis=-1)
    assert (err <= best * (1 + 1e-6) + 1e-12).all()
    assert (np.abs(O.widen_fp8_e4m3(codes)).max(axis=(0, 2)) == 448.0).all()
    deq = O.dequantised_keys(codes, scale)
    assert np.abs(deq - I.bf16_bits_to_f64(bits)).max() <= 20.0 * 5 / 16      # 3 mantissa bits: relative step 1/8

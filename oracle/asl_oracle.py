"""fp64 CPU oracle for the ASL prefill hot path  --  TEST INFRASTRUCTURE ONLY.

A plain, slow, step-by-step numpy restatement of the paper's two algorithms
(Algorithm 1 "GetRanks", Algorithm 2 "SelectTokens") and of the formulas of
Section 4.1 (pooled attention, scores, top(L), var_top, relative variance).
It shares no code, header, table or helper with the CUDA path and never
imports it; only tests, the smoke check and the benchmark's CPU-baseline leg
may call it.  Inputs are bf16 bit patterns widened exactly to float64.

Every function is pinned by tests that do not re-type its formula: closed
forms, invariants, brute force on tiny inputs and library cross-checks
(tests/test_oracle_*.py).  The paper prints no worked numeric example of this
path, so the absolute level of the variance statistic is pinned only by its
closed forms (reversed ranks, identical rows, random permutations) and by
brute force with Python sets.

Readings taken where the paper leaves a choice (each also listed in the
design notes):
  * softmax runs over all n keys, window keys included under the causal mask
    of the last w x w block; only past columns [0, n-w) are kept (Alg. 1 (window softmax A, past-only column sum U));
  * pooling is stride 1, pad floor(S/2); average pooling pads with zeros and
    always divides by S; max pooling looks at in-range taps only (Alg. 1 (1-D pooling));
  * pooling runs per query head, then heads of a GQA group are summed (Alg. 1:
    pooling, then SumGroups); the rank statistic orders tokens by the sum over all heads (Sec. 4.1);
  * ranks are 0-based, descending score, ties to the lower index (stable);
  * the statistic uses the latest L_obs rank rows (Alg. 2 (stacked rank rows R)), population
    variance of raw ranks, mean over the union of per-row top-k sets;
  * top-k ties go to the lower index; kept indices are emitted ascending with
    the window indices appended (Alg. 1 (k, TopK and window append)).
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np

POOL_AVG = 0
POOL_MAX = 1


def widen_bf16(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64, exactly."""
    u32 = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u32.view(np.float32).astype(np.float64)


def widen_fp8_e4m3(codes: np.ndarray) -> np.ndarray:
    """FP8 E4M3 bit patterns (uint8; the "finite" variant of the OCP 8-bit format: one sign bit, four
    exponent bits with bias 7, three mantissa bits, no infinities, S.1111.111 = NaN) -> float64, exactly.
    A quantised K cache stores these codes with one fp32 scale per kv head; the keys the method sees
    are code value x scale (Algorithm 1 takes K as given)."""
    c = np.ascontiguousarray(codes, dtype=np.uint8).astype(np.int64)
    sign = np.where(c & 0x80, -1.0, 1.0)
    e = (c >> 3) & 0xF
    m = (c & 0x7).astype(np.float64)
    normal = np.ldexp(1.0 + m / 8.0, (e - 7).astype(np.int64))
    subnormal = np.ldexp(m / 8.0, -6)
    v = sign * np.where(e == 0, subnormal, normal)
    return np.where((c & 0x7F) == 0x7F, np.nan, v)


def dequantised_keys(codes: np.ndarray, k_scale: np.ndarray) -> np.ndarray:
    """Keys of a quantised cache: codes [n][H_k][d] x one scale per kv head, in float64."""
    return widen_fp8_e4m3(codes) * np.asarray(k_scale, dtype=np.float64)[None, :, None]


# --------------------------------------------------------------------------
# Algorithm 1: window softmax A and the past-only column sum U
# --------------------------------------------------------------------------
def window_attention(q_head: np.ndarray, k_head: np.ndarray) -> np.ndarray:
    """A = Softmax(Q[n-w:n] K^T / sqrt(d) + CausalMaskOnLastBlock(w)) for one
    query head (Alg. 1 (window softmax A); Sec. 4.1 "PA").

    q_head [w][d], k_head [n][d], float64.  Row t sits at position n-w+t and
    sees keys j <= n-w+t.  Returns A [w][n]."""
    w, d = q_head.shape
    n = k_head.shape[0]
    T = n - w
    s = (q_head @ k_head.T) / math.sqrt(d)
    j = np.arange(n)[None, :]
    t = np.arange(w)[:, None]
    s = np.where(j <= T + t, s, -np.inf)
    s = s - s.max(axis=1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=1, keepdims=True)


def window_lse(q_obs: np.ndarray, k: np.ndarray, group: int) -> np.ndarray:
    """lse[a][t] = log of the softmax denominator of window row t of query head a:
    log sum over the visible keys j <= n-w+t of exp(q.k_j / sqrt(d)) (Alg. 1 (window softmax A);
    the quantity a fused attention forward keeps per row).  Returns [H_q][w]."""
    Hq, w, d = q_obs.shape
    n = k.shape[0]
    T = n - w
    out = np.empty((Hq, w), dtype=np.float64)
    for a in range(Hq):
        s = (q_obs[a] @ k[:, a // group, :].T) / math.sqrt(d)
        for t in range(w):
            row = s[t, :T + t + 1]
            m = row.max()
            out[a, t] = m + math.log(np.exp(row - m).sum())
    return out


def past_column_sums(q_obs: np.ndarray, k: np.ndarray, group: int,
                     return_window_mass: bool = False):
    """U[a][j] = sum_t A[a][t][j] for past columns j < n-w (Alg. 1 (past-only column sum U)).

    q_obs [H_q][w][d], k [n][H_k][d], float64; query head a reads kv head
    a // group (contiguous groups, the Reshape([B,H_k,G,.]) of Alg. 1 (SumGroups)).
    Returns U [H_q][n-w]; optionally also the mass that fell on the window's
    own columns, [H_q], so that U.sum + window mass = w per head."""
    Hq, w, d = q_obs.shape
    n = k.shape[0]
    T = n - w
    U = np.empty((Hq, T), dtype=np.float64)
    wm = np.empty(Hq, dtype=np.float64)
    for a in range(Hq):
        A = window_attention(q_obs[a], k[:, a // group, :])
        U[a] = A[:, :T].sum(axis=0)
        wm[a] = A[:, T:].sum()
    return (U, wm) if return_window_mass else U


# --------------------------------------------------------------------------
# Algorithm 1: 1-D pooling, kernel S, stride 1, pad floor(S/2)
# --------------------------------------------------------------------------
def pool1d(U: np.ndarray, S: int, mode: int = POOL_AVG) -> np.ndarray:
    """Pool every row of U [rows][T] along the token axis.

    Average: zero padding, divisor always S.  Max: only in-range taps."""
    if S < 1 or S % 2 == 0:
        raise ValueError("pool kernel must be odd and >= 1")
    rows, T = U.shape
    r = S // 2
    out = np.empty_like(U)
    for j in range(T):
        lo, hi = max(0, j - r), min(T, j + r + 1)
        if mode == POOL_AVG:
            out[:, j] = U[:, lo:hi].sum(axis=1) / S
        else:
            out[:, j] = U[:, lo:hi].max(axis=1)
    return out


# --------------------------------------------------------------------------
# Algorithm 1: SumGroups, and the "scores" formula of Section 4.1
# --------------------------------------------------------------------------
def sum_groups(Vp: np.ndarray, group: int) -> np.ndarray:
    """P[h] = sum_{g<G} Vp[h*G + g]  (Alg. 1 (SumGroups))."""
    Hq, T = Vp.shape
    return Vp.reshape(Hq // group, group, T).sum(axis=1)


def aggregate_scores(P: np.ndarray) -> np.ndarray:
    """scores = sum over groups and heads of the pooled attention (Sec. 4.1)."""
    return P.sum(axis=0)


def score_layer(q_obs: np.ndarray, k: np.ndarray, group: int, S: int, mode: int = POOL_AVG):
    """Alg. 1 from the window softmax to SumGroups for one request.  Returns (P [H_k][T], agg [T])."""
    U = past_column_sums(q_obs, k, group)
    P = sum_groups(pool1d(U, S, mode), group)
    return P, aggregate_scores(P)


# --------------------------------------------------------------------------
# Algorithm 1: RankDesc
# --------------------------------------------------------------------------
def rank_desc(scores: np.ndarray) -> np.ndarray:
    """rank[j] = 0-based position of token j when tokens are ordered by score
    descending, equal scores by index ascending."""
    T = scores.shape[0]
    order = np.lexsort((np.arange(T), -scores))     # last key is primary
    rank = np.empty(T, dtype=np.int64)
    rank[order] = np.arange(T)
    return rank


# --------------------------------------------------------------------------
# Algorithm 2: union of per-layer top-k (J, U), variance of ranks (RelNormVar)
# --------------------------------------------------------------------------
def rank_statistic(R: np.ndarray, k: int) -> Tuple[int, int, float]:
    """R [rows][T] integer rank rows of the latest layers (Alg. 2 (stacked rank rows R)).

    J = the k smallest ranks of each row (TopKIndices), U = Unique(Flatten(J))
    = {j : some row has R[r][j] < k}; var_top = mean over U of the
    population variance over rows of R[:, j] (Sec. 4.1 "var_top").
    Returns (num, m, var_top) with num = sum_{j in U} (rows*sum r^2 - (sum r)^2)
    as an exact integer, m = |U|, var_top = num / (rows^2 * m)."""
    rows, T = R.shape
    in_union = (R < k).any(axis=0)
    m = int(in_union.sum())
    if m == 0:
        return 0, 0, float("nan")
    num = 0
    for j in np.nonzero(in_union)[0]:
        col = [int(x) for x in R[:, j]]
        num += rows * sum(x * x for x in col) - sum(col) ** 2
    return num, m, num / (rows * rows * m)


class SelectionController:
    """Algorithm 2 as a per-layer state machine for one request.

    Holds the rank cache (latest L_obs rows) and init_var.  ``step`` is called
    once per scored layer with that layer's aggregate scores."""

    def __init__(self, budget: int, window: int, l_min: int, l_obs: int, tau: float):
        self.budget, self.window = budget, window
        self.l_min, self.l_obs, self.tau = l_min, l_obs, tau
        self.cache: List[Tuple[int, np.ndarray]] = []
        self.init_var: Optional[float] = None
        self.selected_layer = -1

    def step(self, layer_idx: int, agg: np.ndarray) -> dict:
        T = agg.shape[0]
        self.cache.append((layer_idx, rank_desc(agg)))          # Alg. 1 (RankDesc)
        self.cache = self.cache[-self.l_obs:]
        out = {"layer": layer_idx, "evaluated": False, "selected": False}
        if layer_idx < self.l_min or len(self.cache) < 2:        # Alg. 2 (early return)
            return out
        R = np.stack([r for _, r in self.cache])                 # stacked rank rows R
        k = min(self.budget - self.window, T)                    # k
        num, m, var_top = rank_statistic(R, k)                   # J, U, RelNormVar
        if self.init_var is None:
            self.init_var = var_top
        rel = var_top / self.init_var if self.init_var != 0 else float("nan")
        sel = bool(rel < self.tau)                               # threshold test
        out.update(evaluated=True, rows=R.shape[0], num=num, m=m, var_top=var_top,
                   rel=rel, selected=sel)
        if sel and self.selected_layer < 0:
            self.selected_layer = layer_idx
        return out


# --------------------------------------------------------------------------
# Algorithm 1: k, per-head TopK, window append, and the gather K[I], V[I]
# --------------------------------------------------------------------------
def kept_count(budget: int, n: int, window: int) -> int:
    """k = min(KV_budget, N_q) - W  (Alg. 1 (k))."""
    return min(budget, n) - window


def select_topk(P_row: np.ndarray, k: int, n: int, window: int) -> np.ndarray:
    """I = Concat(TopK(P, k), I_w) for one (request, kv head) (Alg. 1 (TopK and window append)).

    The k past tokens with the largest score, ties to the lower index, listed
    in ascending index order, followed by the window indices n-w .. n-1."""
    T = P_row.shape[0]
    order = np.lexsort((np.arange(T), -P_row))
    top = np.sort(order[:k])
    return np.concatenate([top, np.arange(n - window, n)]).astype(np.int64)


def compact_rows(x: np.ndarray, idx: np.ndarray, head: int) -> np.ndarray:
    """K[I] (or V[I]) for one kv head: rows of x [n][H_k][d] at idx (Alg. 1 (K[I], V[I])).
    Works on any dtype; used on the raw bf16 bit patterns."""
    return x[idx, head, :]


# --------------------------------------------------------------------------
# Algorithm 2: one-shot token selection at the selection layer
# --------------------------------------------------------------------------
def select_tokens(agg: np.ndarray, budget: int, n: int, window: int) -> np.ndarray:
    """select_idx = Unique(J_last u I_w) (Alg. 2 (one-shot selection)): J_last are the k tokens with the
    smallest rank of the current layer, i.e. the k best aggregate scores (ties to the lower
    index), I_w the window tokens T .. T+W-1; Unique sorts.  k = min(budget - W, T)."""
    T = agg.shape[0]
    k = min(budget - window, T)
    rank = rank_desc(agg)
    J_last = np.nonzero(rank < k)[0]
    I_w = np.arange(T, T + window)
    return np.unique(np.concatenate([J_last, I_w])).astype(np.int64)

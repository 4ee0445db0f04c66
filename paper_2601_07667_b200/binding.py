"""ctypes binding of libasl_b200.so: same names as the C ABI, argument
marshalling only.  Every step of the path runs in the library's CUDA kernels;
PyTorch supplies device memory and streams, nothing else.  There is no CPU
fallback: a missing library is an ImportError, a failing call an AslError."""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libasl_b200.so")

ASL_POOL_AVG, ASL_POOL_MAX = 0, 1
ASL_K_BF16, ASL_K_FP8_E4M3 = 0, 1
ASL_OK, ASL_ERR_INVALID, ASL_ERR_UNSUPPORTED, ASL_ERR_WORKSPACE = 0, -1, -2, -3
ASL_ERR_CUDA, ASL_ERR_TIMEOUT, ASL_ERR_ARCH = -4, -5, -6

EXPORTS = ("asl_create", "asl_destroy", "asl_plan", "asl_plan_sizes", "asl_score_layer", "asl_rank_stat",
           "asl_select_topk", "asl_compact_kv", "asl_device_status", "asl_launch_count", "asl_strerror",
           "asl_rank_desc_static", "asl_score_layer_lse", "asl_window_lse", "asl_compact_rows",
           "asl_score_columns", "asl_pool_scores", "asl_set_controller", "asl_select_topk_gated",
           "asl_selftest_bounded_wait", "asl_set_layer")
ASL_RANK_STATIC_MAX_T = 262144


class AslParams(C.Structure):
    _fields_ = [("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("window", C.c_int32), ("pool_kernel", C.c_int32), ("pool_mode", C.c_int32),
                ("batch", C.c_int32), ("l_min", C.c_int32), ("l_obs", C.c_int32), ("score_ctas", C.c_int32),
                ("tau", C.c_double),
                ("cu_seqlens", C.POINTER(C.c_int32)), ("budgets", C.POINTER(C.c_int32)),
                ("q_stride", C.c_int64 * 3), ("k_stride", C.c_int64 * 2), ("v_stride", C.c_int64 * 2),
                ("k_dtype", C.c_int32), ("reserved0", C.c_int32), ("k_scale", C.POINTER(C.c_float))]


class AslStat(C.Structure):
    _fields_ = [("num", C.c_int64), ("m", C.c_int32), ("rows", C.c_int32), ("k", C.c_int32),
                ("layer_idx", C.c_int32), ("evaluated", C.c_int32), ("selected", C.c_int32),
                ("has_init", C.c_int32), ("reserved", C.c_int32),
                ("var_top", C.c_double), ("init_var", C.c_double), ("rel", C.c_double)]


STAT_DTYPE = np.dtype([("num", "<i8"), ("m", "<i4"), ("rows", "<i4"), ("k", "<i4"), ("layer_idx", "<i4"),
                       ("evaluated", "<i4"), ("selected", "<i4"), ("has_init", "<i4"), ("reserved", "<i4"),
                       ("var_top", "<f8"), ("init_var", "<f8"), ("rel", "<f8")])
assert STAT_DTYPE.itemsize == C.sizeof(AslStat) == 64


class AslError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: {asl_strerror(status)} ({status})")


def _load() -> C.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2601_07667_b200.build` "
                          "(there is no CPU fallback)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    lib.asl_create.argtypes = [C.POINTER(vp), C.c_int]
    lib.asl_destroy.argtypes = [vp]
    lib.asl_plan.argtypes = [vp, C.POINTER(AslParams), C.POINTER(sz)]
    lib.asl_plan_sizes.argtypes = [vp, C.POINTER(i64), C.POINTER(i64), C.POINTER(i64)]
    lib.asl_score_layer.argtypes = [vp, vp, vp, vp, vp, vp, sz, vp]
    lib.asl_score_layer_lse.argtypes = [vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.asl_window_lse.argtypes = [vp, vp, sz, vp, vp]
    lib.asl_set_controller.argtypes = [vp, i32]
    lib.asl_set_layer.argtypes = [vp, i32]
    lib.asl_select_topk_gated.argtypes = [vp, vp, i32, vp, vp, i32, vp, sz, vp]
    lib.asl_score_columns.argtypes = [vp, vp, vp, vp, vp, sz, i32, vp]
    lib.asl_pool_scores.argtypes = [vp, vp, sz, i32, vp, vp, vp]
    lib.asl_compact_rows.argtypes = [vp, vp, vp, vp, i64, vp]
    lib.asl_rank_stat.argtypes = [vp, vp, i32, i32, vp, vp, vp, sz, vp]
    lib.asl_select_topk.argtypes = [vp, vp, i32, vp, vp, sz, vp]
    lib.asl_compact_kv.argtypes = [vp, vp, vp, vp, vp, vp, vp]
    lib.asl_device_status.argtypes = [vp, vp, C.POINTER(i32)]
    lib.asl_rank_desc_static.argtypes = [vp, i32, vp, vp]
    lib.asl_selftest_bounded_wait.argtypes = [vp, i32, i64, vp]
    lib.asl_launch_count.argtypes = [vp]
    lib.asl_launch_count.restype = i64
    lib.asl_strerror.argtypes = [C.c_int]
    lib.asl_strerror.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("asl_launch_count", "asl_strerror"):
            getattr(lib, name).restype = C.c_int
    return lib


_lib = _load()


def library() -> C.CDLL:
    return _lib


def asl_strerror(status: int) -> str:
    return _lib.asl_strerror(int(status)).decode()


def _check(status: int, what: str) -> None:
    if status != ASL_OK:
        raise AslError(status, what)


def _ptr(x) -> int:
    """Device (or host) address of a torch tensor / raw integer address."""
    if x is None:
        return 0
    if isinstance(x, int):
        return x
    return x.data_ptr()


def _stream_handle(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


# ---- the C entry points, one Python function each ---------------------------------
def asl_create(device: int = 0) -> int:
    h = C.c_void_p()
    _check(_lib.asl_create(C.byref(h), int(device)), "asl_create")
    return h.value


def asl_destroy(ctx: int) -> None:
    _check(_lib.asl_destroy(ctx), "asl_destroy")


def asl_plan(ctx: int, *, n_q_heads: int, n_kv_heads: int, head_dim: int, window: int, pool_kernel: int,
             pool_mode: int, cu_seqlens: Sequence[int], budgets: Sequence[int], l_min: int, l_obs: int,
             tau: float, q_stride: Sequence[int], k_stride: Sequence[int], v_stride: Sequence[int],
             score_ctas: int = 0, k_dtype: int = ASL_K_BF16, k_scale: Optional[Sequence[float]] = None) -> int:
    cu = (C.c_int32 * len(cu_seqlens))(*[int(x) for x in cu_seqlens])
    bu = (C.c_int32 * len(budgets))(*[int(x) for x in budgets])
    ks = (C.c_float * len(k_scale))(*[float(x) for x in k_scale]) if k_scale is not None else None
    p = AslParams(n_q_heads, n_kv_heads, head_dim, window, pool_kernel, pool_mode, len(budgets), l_min, l_obs, int(score_ctas),
                  float(tau), cu, bu, (C.c_int64 * 3)(*q_stride), (C.c_int64 * 2)(*k_stride),
                  (C.c_int64 * 2)(*v_stride), int(k_dtype), 0, ks)
    if k_scale is not None and len(k_scale) != n_kv_heads:
        raise AslError(ASL_ERR_INVALID, "asl_plan")
    if len(cu_seqlens) != len(budgets) + 1:
        raise AslError(ASL_ERR_INVALID, "asl_plan")
    size = C.c_size_t(0)
    _check(_lib.asl_plan(ctx, C.byref(p), C.byref(size)), "asl_plan")
    return size.value


def asl_plan_sizes(ctx: int):
    a, b, c = C.c_int64(), C.c_int64(), C.c_int64()
    _check(_lib.asl_plan_sizes(ctx, C.byref(a), C.byref(b), C.byref(c)), "asl_plan_sizes")
    return a.value, b.value, c.value


def asl_score_layer(ctx, q_obs, k, scores_kv, scores_agg, workspace, workspace_bytes, stream=None) -> None:
    _check(_lib.asl_score_layer(ctx, _ptr(q_obs), _ptr(k), _ptr(scores_kv), _ptr(scores_agg), _ptr(workspace),
                                int(workspace_bytes), _stream_handle(stream)), "asl_score_layer")


def asl_score_layer_lse(ctx, q_obs, k, lse, scores_kv, scores_agg, workspace, workspace_bytes, stream=None) -> None:
    _check(_lib.asl_score_layer_lse(ctx, _ptr(q_obs), _ptr(k), _ptr(lse), _ptr(scores_kv), _ptr(scores_agg),
                                    _ptr(workspace), int(workspace_bytes), _stream_handle(stream)), "asl_score_layer_lse")


ASL_CONTROLLER_REPORT, ASL_CONTROLLER_LATCH = 0, 1


def asl_set_controller(ctx, mode: int) -> None:
    _check(_lib.asl_set_controller(ctx, int(mode)), "asl_set_controller")


def asl_set_layer(ctx, layer_idx: int) -> None:
    _check(_lib.asl_set_layer(ctx, int(layer_idx)), "asl_set_layer")


def asl_select_topk_gated(ctx, scores, n_heads, idx_out, stat, layer_idx, workspace, workspace_bytes, stream=None) -> None:
    _check(_lib.asl_select_topk_gated(ctx, _ptr(scores), int(n_heads), _ptr(idx_out), _ptr(stat), int(layer_idx),
                                      _ptr(workspace), int(workspace_bytes), _stream_handle(stream)),
           "asl_select_topk_gated")


def asl_score_columns(ctx, q_obs, k, lse, workspace, workspace_bytes, slot, stream=None) -> None:
    _check(_lib.asl_score_columns(ctx, _ptr(q_obs), _ptr(k), _ptr(lse), _ptr(workspace), int(workspace_bytes), int(slot),
                                  _stream_handle(stream)), "asl_score_columns")


def asl_pool_scores(ctx, workspace, workspace_bytes, slot, scores_kv, scores_agg, stream=None) -> None:
    _check(_lib.asl_pool_scores(ctx, _ptr(workspace), int(workspace_bytes), int(slot), _ptr(scores_kv), _ptr(scores_agg),
                                _stream_handle(stream)), "asl_pool_scores")


def asl_window_lse(ctx, workspace, workspace_bytes, lse_out, stream=None) -> None:
    _check(_lib.asl_window_lse(ctx, _ptr(workspace), int(workspace_bytes), _ptr(lse_out), _stream_handle(stream)),
           "asl_window_lse")


def asl_rank_stat(ctx, scores_agg, layer_idx, n_rows, rank_ring, stat, workspace, workspace_bytes, stream=None) -> None:
    _check(_lib.asl_rank_stat(ctx, _ptr(scores_agg), int(layer_idx), int(n_rows), _ptr(rank_ring), _ptr(stat),
                              _ptr(workspace), int(workspace_bytes), _stream_handle(stream)), "asl_rank_stat")


def asl_select_topk(ctx, scores, n_heads, idx_out, workspace, workspace_bytes, stream=None) -> None:
    _check(_lib.asl_select_topk(ctx, _ptr(scores), int(n_heads), _ptr(idx_out), _ptr(workspace),
                                int(workspace_bytes), _stream_handle(stream)), "asl_select_topk")


def asl_compact_kv(ctx, k, v, idx, k_out, v_out, stream=None) -> None:
    _check(_lib.asl_compact_kv(ctx, _ptr(k), _ptr(v), _ptr(idx), _ptr(k_out), _ptr(v_out),
                               _stream_handle(stream)), "asl_compact_kv")


def asl_compact_rows(ctx, x, idx, out, row_bytes, stream=None) -> None:
    _check(_lib.asl_compact_rows(ctx, _ptr(x), _ptr(idx), _ptr(out), int(row_bytes), _stream_handle(stream)),
           "asl_compact_rows")


def asl_device_status(ctx, stream=None):
    where = C.c_int32(0)
    st = _lib.asl_device_status(ctx, _stream_handle(stream), C.byref(where))
    return st, where.value


def asl_selftest_bounded_wait(ctx, which: int, limit_ns: int, stream=None) -> None:
    _check(_lib.asl_selftest_bounded_wait(ctx, int(which), int(limit_ns), _stream_handle(stream)),
           "asl_selftest_bounded_wait")


def asl_launch_count(ctx) -> int:
    return int(_lib.asl_launch_count(ctx))


def asl_rank_desc_static(scores, T: int, rank_out, stream=None) -> None:
    """Rank row of one request's scores with no context, no workspace and no
    allocation: for callers that may not allocate device memory when they need
    it (a server whose pool is owned by its own allocator, code inside another
    runtime's callback).  The sort scratch is a fixed array inside the library,
    shared by every call on the device, so calls that could overlap on the GPU
    must be ordered; T is limited to ASL_RANK_STATIC_MAX_T."""
    _check(_lib.asl_rank_desc_static(_ptr(scores), int(T), _ptr(rank_out), _stream_handle(stream)),
           "asl_rank_desc_static")


# ---- a small holder of one plan's device buffers -------------------------------------
class LayerPath:
    """Owns a context, its plan and the device buffers of one layer's pass
    (scores, indices, compacted cache, rank ring, statistic), all torch tensors.
    ``run_layer`` issues the five steps: the scoring proper on the current stream, the
    rest of the layer (pooling first) on a side stream (``tail_streams=2``: pooling and the rank
    statistic on one, top-k and compaction on another) that is not waited for, so that it overlaps the scoring of the next layer (both
    score buffers are double buffered for that; give the plan ``score_ctas``
    below the SM count to leave those kernels somewhere to run).  ``join`` makes
    the current stream wait for everything issued so far; ``read_stat`` joins by
    itself.  A device-wide synchronize covers it too."""

    def __init__(self, *, n_q_heads, n_kv_heads, head_dim, window, pool_kernel, pool_mode, seqlens, budgets,
                 l_min, l_obs, tau, device: int = 0, q_stride=None, k_stride=None, v_stride=None,
                 score_ctas: int = 0, tail_streams: int = 1, k_dtype: int = ASL_K_BF16, k_scale=None):
        import torch
        self.torch = torch
        self.dev = torch.device("cuda", device)
        self.ctx = asl_create(device)
        self.H_q, self.H_k, self.d, self.w = n_q_heads, n_kv_heads, head_dim, window
        self.l_min, self.l_obs = l_min, l_obs
        self.seqlens = [int(n) for n in seqlens]
        self.batch = len(self.seqlens)
        cu = np.concatenate([[0], np.cumsum(self.seqlens)]).astype(np.int64)
        self.cu = cu
        q_stride = q_stride or (n_q_heads * window * head_dim, window * head_dim, head_dim)
        k_stride = k_stride or (n_kv_heads * head_dim, head_dim)
        v_stride = v_stride or (n_kv_heads * head_dim, head_dim)
        self.ws_bytes = asl_plan(self.ctx, n_q_heads=n_q_heads, n_kv_heads=n_kv_heads, head_dim=head_dim,
                                 window=window, pool_kernel=pool_kernel, pool_mode=pool_mode, cu_seqlens=cu,
                                 budgets=budgets, l_min=l_min, l_obs=l_obs, tau=tau, q_stride=q_stride,
                                 k_stride=k_stride, v_stride=v_stride, score_ctas=score_ctas, k_dtype=k_dtype,
                                 k_scale=k_scale)
        self.sum_tokens, self.sum_T, self.sum_kept = asl_plan_sizes(self.ctx)
        self.kept = [min(int(bg), n) for bg, n in zip(budgets, self.seqlens)]
        self.t_off = np.concatenate([[0], np.cumsum([n - window for n in self.seqlens])]).astype(np.int64)
        self.kept_off = np.concatenate([[0], np.cumsum(self.kept)]).astype(np.int64)
        dev = self.dev
        self.workspace = torch.empty(max(self.ws_bytes, 256), dtype=torch.uint8, device=dev)
        self._kv = [torch.empty((n_kv_heads, self.sum_T), dtype=torch.float32, device=dev) for _ in range(2)]
        self._agg = [torch.empty((self.sum_T,), dtype=torch.float32, device=dev) for _ in range(2)]
        self._agg_free = [None, None]       # event after the side-stream work that last read the buffers
        self._cur = 0
        self.idx = torch.empty((n_kv_heads, self.sum_kept), dtype=torch.int32, device=dev)
        self.k_out = torch.empty((n_kv_heads, self.sum_kept, head_dim),
                                 dtype=torch.uint8 if k_dtype == ASL_K_FP8_E4M3 else torch.bfloat16, device=dev)
        self.v_out = torch.empty((n_kv_heads, self.sum_kept, head_dim), dtype=torch.bfloat16, device=dev)
        self.rank_ring = torch.zeros((l_obs, self.sum_T), dtype=torch.int32, device=dev)
        self.stat = torch.zeros((self.batch, C.sizeof(AslStat)), dtype=torch.uint8, device=dev)
        self.side = torch.cuda.Stream(device=dev)       # rank statistic
        self.side2 = torch.cuda.Stream(device=dev) if tail_streams >= 2 else self.side     # top-k and compaction
        self._fork = torch.cuda.Event()
        self._join = torch.cuda.Event()
        self._join2 = torch.cuda.Event()
        self.first_layer: Optional[int] = None
        self.latch = False

    def set_controller(self, mode: int) -> None:
        """ASL_CONTROLLER_LATCH: selections are final on the device and ``run_layer`` tells the library the
        layer of its calls, so that the work of finished requests is skipped."""
        asl_set_controller(self.ctx, mode)
        self.latch = mode == ASL_CONTROLLER_LATCH

    @property
    def scores_kv(self):
        """Per-kv-head scores of the latest layer (device fp32 [H_k][sum_T])."""
        return self._kv[self._cur]

    @property
    def scores_agg(self):
        """Aggregate scores of the latest layer (device fp32 [sum_T])."""
        return self._agg[self._cur]

    def _fresh_events(self) -> None:
        torch = self.torch
        self._agg_free = [None, None]
        self._fork, self._join, self._join2 = torch.cuda.Event(), torch.cuda.Event(), torch.cuda.Event()

    def capture(self, steps):
        """Records ``run_layer`` for every ``(q_obs, k, v, layer_idx)`` (or ``(..., lse)``) of ``steps``,
        followed by ``join``, into one CUDA graph and returns it (a ``torch.cuda.CUDAGraph``):
        ``replay()`` then issues the whole sequence - the side streams included - as a single
        launch, which removes the host's per-launch cost and shortens the gaps between the
        dependent kernels of the statistic and the top-k.  The tensors must stay alive and in
        place; run the same steps once without the graph first (module loading, lazy set-up)."""
        torch = self.torch
        torch.cuda.synchronize(self.dev)
        self._fresh_events()            # nothing recorded outside the capture may be waited for inside it
        graph = torch.cuda.CUDAGraph()
        # thread_local: calls that other host threads make meanwhile (a process group's watchdog,
        # a clock sampler) neither end up in the graph nor invalidate the capture
        with torch.cuda.graph(graph, capture_error_mode="thread_local"):
            for step in steps:
                q_obs, k, v, layer_idx = step[:4]
                self.run_layer(q_obs, k, v, layer_idx, lse=step[4] if len(step) > 4 else None)
            self.join()
        self._fresh_events()            # and nothing recorded inside it afterwards
        return graph

    def join(self) -> None:
        """The current stream waits for the statistic work issued so far."""
        cur = self.torch.cuda.current_stream()
        cur.wait_event(self._join)
        cur.wait_event(self._join2)

    def close(self) -> None:
        if self.ctx:
            asl_destroy(self.ctx)
            self.ctx = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self) -> None:
        """New prompt: forget init_var and the rank rows."""
        self.stat.zero_()
        self.first_layer = None

    def n_rows(self, layer_idx: int) -> int:
        if self.first_layer is None:
            self.first_layer = layer_idx
        return min(self.l_obs, layer_idx - self.first_layer + 1)

    def run_layer(self, q_obs, k, v, layer_idx: int, *, overlap: bool = True, score_marks=None, lse=None) -> None:
        """Steps a1..a5 for one layer on the current stream; with ``overlap`` the statistic
        runs on the side stream and is left in flight (see ``join``).  ``score_marks``: a list
        that receives a (start, end) event pair around the scoring call."""
        torch = self.torch
        ctx, ws, wsb = self.ctx, self.workspace, self.ws_bytes
        rows = self.n_rows(layer_idx)
        main = torch.cuda.current_stream()
        if self.latch:
            asl_set_layer(ctx, layer_idx)
        self._cur ^= 1
        agg, skv = self._agg[self._cur], self._kv[self._cur]
        if self._agg_free[self._cur] is not None:
            for done in self._agg_free[self._cur]:          # the side work of two layers ago has read them
                main.wait_event(done)
        if score_marks is not None:
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(main)
        asl_score_columns(ctx, q_obs, k, lse, ws, wsb, self._cur)      # lse: the window rows' log-sum-exp, or None
        if score_marks is not None:
            e1.record(main)
            score_marks.append((e0, e1))
        if overlap:
            self._fork.record(main)
            self.side.wait_event(self._fork)
        asl_pool_scores(ctx, ws, wsb, self._cur, skv, agg, self.side if overlap else main)
        if overlap and self.side2 is not self.side:
            pooled = torch.cuda.Event()
            pooled.record(self.side)
            self.side2.wait_event(pooled)
        s1, s2 = (self.side, self.side2) if overlap else (main, main)
        asl_rank_stat(ctx, agg, layer_idx, rows, self.rank_ring, self.stat, ws, wsb, s1)
        asl_select_topk(ctx, skv, self.H_k, self.idx, ws, wsb, s2)
        asl_compact_kv(ctx, k, v, self.idx, self.k_out, self.v_out, s2)
        if overlap:
            d1, d2 = torch.cuda.Event(), torch.cuda.Event()
            d1.record(self.side)
            d2.record(self.side2)
            self._agg_free[self._cur] = (d1, d2)
            self._join.record(self.side)
            self._join2.record(self.side2)

    def read_stat(self) -> np.ndarray:
        """Device -> host copy of the [B] statistic records (synchronises)."""
        self.join()
        return self.stat.cpu().numpy().view(STAT_DTYPE).reshape(self.batch)

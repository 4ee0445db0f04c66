"""GPU parity at the benchmark's full sizes (the five named workloads).  The sweeps run in the
library's default launch configuration (one scorer CTA per SM, one side stream); the
``benched_launch`` tests repeat the long-context and the ragged workload in the configuration
bench.py times (fewer scorer CTAs, two side streams), issued call by call and replayed from CUDA
graphs.  The oracle computes whole layers here (seconds each on the host), so the comparison stays
element by element; the number of layers is bounded to keep the suite within minutes."""
import numpy as np
import pytest
import torch

from paper_2601_07667_b200 import inputs as I

from asl_check import StatReplay, bench_launch, check_layer, make_path, oracle_layer, to_dev, verify_layer

pytestmark = pytest.mark.gpu


def sweep(wl, seed, layers):
    path = make_path(wl)
    replay = StatReplay(wl)
    rel_gpu, rel_ref = {}, {}
    for layer in layers:
        x = I.layer_inputs(wl, layer, seed)
        res = check_layer(path, wl, x, layer)
        iso, e2e = replay.step(path, layer, res)[0]
        if iso["evaluated"]:
            rel_gpu[layer], rel_ref[layer] = iso["rel"], e2e["rel"]
    sel_gpu = [c.selected_layer for c in replay.on_gpu_scores]
    sel_ref = [c.selected_layer for c in replay.on_ref_scores]
    path.close()
    return rel_gpu, rel_ref, sel_gpu, sel_ref


def test_c2_layer_sweep_selects_the_same_layer():
    wl = I.workload("C2")
    first = wl.l_min - wl.l_obs + 1                        # ring is full when the statistic starts
    rel_gpu, rel_ref, sel_gpu, sel_ref = sweep(wl, 0, range(first, wl.layers))
    assert sel_gpu == sel_ref
    assert first < sel_ref[0] < wl.layers - 1               # crosses the threshold mid-stack
    ls = sorted(rel_ref)
    assert min(ls, key=lambda l: rel_gpu[l]) == min(ls, key=lambda l: rel_ref[l])
    dev = max(abs(rel_gpu[l] - rel_ref[l]) for l in ls)
    margin = min(abs(rel_ref[l] - wl.tau) for l in ls)
    assert margin >= 10 * dev, f"threshold margin {margin:.4f} vs GPU/oracle deviation {dev:.5f}"


def test_c3_long_context_layers():
    wl = I.workload("C3")
    rel_gpu, rel_ref, sel_gpu, sel_ref = sweep(wl, 0, range(0, 4))
    assert sel_gpu == sel_ref


def test_c4_ragged_batch_full():
    wl = I.workload("C4", seed=0)
    sweep(wl, 0, range(0, 2))


def test_c5_wide_gqa_max_pool_full():
    wl = I.workload("C5")
    sweep(wl, 0, range(0, 2))


def test_half_million_token_context():
    """524352 tokens in one request (8q/2kv so that the oracle still takes seconds): 4097 key tiles per
    segment, 256 rank tiles (the separate scan kernel), 128 top-k tiles, 32-bit offsets near 2^30."""
    wl = I.workload("C3", n_q_heads=8, n_kv_heads=2, seqlens=(524288 + 64,), budgets=(8192,), layers=2, l_min=1,
                    l_obs=2)
    sweep(wl, 3, range(0, 2))


def test_million_token_context():
    """1048640 tokens in one request (8q/2kv): 8193 key tiles per segment, 512 rank tiles, 256 top-k tiles;
    score and token offsets beyond 2^20, packed K rows beyond 2^31 bytes."""
    wl = I.workload("C3", n_q_heads=8, n_kv_heads=2, seqlens=(1048576 + 64,), budgets=(8192,), layers=1, l_min=1,
                    l_obs=2)
    sweep(wl, 4, range(0, 1))


def test_c3_long_context_with_an_fp8_key_cache():
    """The 128K-token workload with K as FP8 (E4M3) codes, in bench.py's launch configuration."""
    from paper_2601_07667_b200 import binding as B
    from asl_check import with_fp8_keys
    wl = I.workload("C3")
    x = with_fp8_keys(I.layer_inputs(wl, 0, 0))
    path = make_path(wl, k_dtype=B.ASL_K_FP8_E4M3, k_scale=[float(s) for s in x["k_scale"]], **bench_launch())
    check_layer(path, wl, x, 0)
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


def _benched_launch_case(wl, seed, n_layers):
    """Layers 0..n_layers-1 in bench.py's launch configuration: call by call, then the same layers
    recorded one per CUDA graph and replayed twice over, every output checked against the oracle
    after each replay."""
    path = make_path(wl, **bench_launch())
    xs = [I.layer_inputs(wl, l, seed) for l in range(n_layers)]
    refs = [oracle_layer(wl, x) for x in xs]
    dev = [(to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])) for x in xs]
    for l in range(n_layers):                                            # (a) call by call
        check_layer(path, wl, xs[l], l, q_dev=dev[l][0], k_dev=dev[l][1], v_dev=dev[l][2], ref=refs[l])
    graphs, cur = [], []
    for l in range(n_layers):                                            # (b) one layer per graph
        graphs.append(path.capture([dev[l] + (l,)]))
        cur.append(path._cur)                                            # score buffer the recorded layer writes
    for _ in range(2):
        for l in range(n_layers):
            graphs[l].replay()
            torch.cuda.synchronize()
            path._cur = cur[l]
            verify_layer(path, wl, xs[l], l, ref=refs[l])
    from paper_2601_07667_b200 import binding as B
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


def test_c3_benched_launch_calls_and_graph_replay():
    _benched_launch_case(I.workload("C3"), 0, 2)


def test_c3_one_pass_step_in_its_benched_launch():
    """The 128K workload scored in one pass from the oracle's log-sum-exp, in the launch configuration
    bench.py times that step in, side streams included: every output against the oracle."""
    from paper_2601_07667_b200 import binding as B
    from asl_check import O
    wl = I.workload("C3")
    x = I.layer_inputs(wl, 0, 0)
    path = make_path(wl, **bench_launch(one_pass=True))
    lse_ref = O.window_lse(O.widen_bf16(x["q_obs"][0]), O.widen_bf16(x["k"]), wl.group)
    lse_dev = torch.from_numpy(lse_ref.astype(np.float32)).cuda().reshape(1, wl.n_q_heads, wl.window)
    q, k, v = to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])
    for _ in range(2):
        path.run_layer(q, k, v, 0, lse=lse_dev)
        path.join()
        torch.cuda.synchronize()
        verify_layer(path, wl, x, 0, check_stat=False)
        path.reset()
    assert B.asl_device_status(path.ctx)[0] == B.ASL_OK
    path.close()


def test_c4_benched_launch_calls_and_graph_replay():
    _benched_launch_case(I.workload("C4", seed=0), 0, 1)


def test_whole_bench_sequence_as_one_graph_matches_the_oracle_on_its_last_layer():
    """The form bench.py replays: several layers, side streams included, in ONE graph."""
    wl = I.workload("C3")
    path = make_path(wl, **bench_launch())
    xs = [I.layer_inputs(wl, l, 0) for l in range(3)]
    dev = [(to_dev(x["q_obs"]), to_dev(x["k"]), to_dev(x["v"])) for x in xs]
    for l in range(3):
        path.run_layer(*dev[l], l)
    graph = path.capture([dev[l] + (l,) for l in range(3)])
    for _ in range(2):
        graph.replay()
        torch.cuda.synchronize()
        verify_layer(path, wl, xs[2], 2)
    path.close()

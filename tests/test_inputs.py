"""The seeded generators: determinism, shapes, planted structure."""
import numpy as np

from paper_2601_07667_b200 import inputs as I


def test_bf16_round_trip_and_rounding():
    x = np.array([1.0, -2.5, 3.14159, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -9], dtype=np.float32)
    bits = I.f32_to_bf16_bits(x)
    back = I.bf16_bits_to_f32(bits)
    assert back[0] == 1.0 and back[1] == -2.5
    assert back[3] == 1.0                      # exactly half way: ties to even
    assert back[4] == np.float32(1.0 + 2 ** -7)
    assert np.abs(back - x).max() <= 2 ** -8 * 4


def test_layers_are_reproducible_and_distinct():
    wl = I.workload("C1", seqlens=(600,), budgets=(100,))
    a = I.layer_inputs(wl, 2, seed=5)
    b = I.layer_inputs(wl, 2, seed=5)
    c = I.layer_inputs(wl, 3, seed=5)
    for key in ("q_obs", "k", "v"):
        assert a[key].dtype == np.uint16 and (a[key] == b[key]).all()
        assert (a[key] != c[key]).any()
    assert a["q_obs"].shape == (1, 8, 32, 128) and a["k"].shape == (600, 2, 128)


def test_planted_keys_are_scaled_copies_of_the_direction():
    wl = I.workload("C1", seqlens=(600,), budgets=(100,))
    x = I.layer_inputs(wl, 0, seed=1)
    u = I.directions(wl, 1)
    pos = I.planted_positions(wl, 1)[0]
    assert pos.shape == (2, 8) and pos.max() < 600 - 32
    k = I.bf16_bits_to_f32(x["k"])
    q = I.bf16_bits_to_f32(x["q_obs"])
    for h in range(2):
        kk = k[pos[h], h, :]
        cos = (kk @ u[0, h]) / np.linalg.norm(kk, axis=1)
        assert (cos > 0.999).all()
        assert np.allclose(np.linalg.norm(kk, axis=1), 3 * np.sqrt(128), rtol=0.01)
    qa = q[0, 5]                                # q head 5 -> kv head 1
    cosq = (qa @ u[0, 1]) / np.linalg.norm(qa, axis=1)
    assert abs(cosq.mean() - 0.5) < 0.05


def test_ragged_workload_shapes():
    wl = I.workload("C4", seed=3)
    assert wl.batch == 8 and all(8192 <= n <= 65536 for n in wl.seqlens)
    assert wl.budgets == tuple(n // 10 for n in wl.seqlens)
    cu = wl.cu_seqlens()
    assert cu[0] == 0 and cu[-1] == wl.total_tokens and cu.dtype == np.int32
    small = I.workload("C4", seqlens=(300, 450), budgets=(40, 50))
    x = I.layer_inputs(small, 0)
    assert x["k"].shape == (750, 8, 128) and x["q_obs"].shape == (2, 32, 32, 128)
    pos = I.planted_positions(small, 0)
    assert pos[0].shape == (8, 1) and pos[1].max() < 450 - 32


def test_distractors_have_the_stated_cosine():
    wl = I.workload("C3", seqlens=(2000,), budgets=(300,))
    x = I.layer_inputs(wl, 0)
    u = I.directions(wl, 0)
    dpos = I.distractor_positions(wl, 0)[0]
    k = I.bf16_bits_to_f32(x["k"])
    kk = k[dpos[3], 3, :]
    cos = (kk @ u[0, 3]) / np.linalg.norm(kk, axis=1)
    assert kk.shape[0] == 64 and np.allclose(cos, 0.9, atol=0.01)


def test_quantised_scores_have_ties():
    s = I.quantised_scores(2, 1000, 16, seed=1)
    assert s.dtype == np.float32 and np.unique(s).size <= 16

"""The allocation-free rank row (asl_rank_desc_static) against the regular entry
point (asl_rank_stat), through the C ABI.

Why the entry point exists: some users of the library cannot allocate device
memory at the moment they need a rank row (their server gave all memory to its
own pool at start-up, or they run inside another runtime's callback), so they
can build neither a context nor a workspace.  The static variant sorts in a
fixed scratch array that lives inside the library and is reused by every call.

The file name sorts last on purpose: a run that stops at the first failure has
then already run every other test.  The checks hold both in a fresh process
and after the rest of the suite, because nothing here depends on what the
scratch array held before: two different inputs of different lengths are ranked
back to back, the second shorter than the first, so stale keys from the first
call sit right behind the second call's data."""
import numpy as np
import pytest
import torch

from oracle import asl_oracle as O
from paper_2601_07667_b200 import inputs as I

from asl_check import make_path

pytestmark = pytest.mark.gpu


def ring_row_by_regular_entry_point(scores: torch.Tensor) -> torch.Tensor:
    """Rank row the context-based asl_rank_stat writes for the same scores."""
    from paper_2601_07667_b200 import binding as B
    T, w = scores.numel(), 32
    wl = I.workload("C1", seqlens=(T + w,), budgets=(w + 1,), l_min=5, l_obs=2)
    path = make_path(wl)
    path.scores_agg.copy_(scores)
    B.asl_rank_stat(path.ctx, path.scores_agg, 0, 1, path.rank_ring, path.stat, path.workspace, path.ws_bytes)
    torch.cuda.synchronize()
    row = path.rank_ring[0].clone()
    path.close()
    return row


def test_static_rank_row_matches_the_regular_one_twice_in_a_row():
    from paper_2601_07667_b200 import binding as B
    g = torch.Generator().manual_seed(11)
    first = torch.randn(70001, generator=g)                                    # several sort tiles + a ragged tail
    second = torch.from_numpy(I.quantised_scores(1, 9000, 5, seed=3)[0])      # shorter, long runs of exact ties
    cases = [first.cuda(), second.cuda()]
    expected = [ring_row_by_regular_entry_point(s) for s in cases]
    outs = [torch.full((s.numel(),), -1, dtype=torch.int32, device="cuda") for s in cases]
    B.asl_rank_desc_static(cases[0], cases[0].numel(), outs[0])               # first call on the device: set-up
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    for s, out in zip(cases, outs):                                            # two calls in a row, same stream
        B.asl_rank_desc_static(s, s.numel(), out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before, "the calls must not take device memory"
    for s, out, ref in zip(cases, outs, expected):
        assert torch.equal(out, ref)                                           # integer work: bit-exact
        # and against the definition itself: the oracle's RankDesc of the same fp32 scores
        assert (out.cpu().numpy() == O.rank_desc(s.cpu().numpy().astype(np.float64))).all()


def test_static_rank_row_refuses_what_it_cannot_hold():
    from paper_2601_07667_b200 import binding as B
    t = torch.zeros(16, dtype=torch.float32, device="cuda")
    o = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(B.AslError) as e:
        B.asl_rank_desc_static(t, B.ASL_RANK_STATIC_MAX_T + 1, o)              # refused before any launch
    assert e.value.status == B.ASL_ERR_WORKSPACE
    for bad in ((None, 16, o), (t, 16, None), (t, 0, o)):
        with pytest.raises(B.AslError) as e:
            B.asl_rank_desc_static(*bad)
        assert e.value.status == B.ASL_ERR_INVALID

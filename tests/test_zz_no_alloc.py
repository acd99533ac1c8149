"""maxscore_index_build_noalloc: the index build for callers that cannot allocate device memory.

Some users of this library run where device allocation is off the table: inside a serving loop where a
cudaMalloc would stall the GPU, as a plugin that may only touch tensors its host framework hands it, or
on top of a pool that is already fully carved up.  For them the library offers one entry point that
needs no context and no workspace; its scratch sits in a fixed array inside the library.  This test
calls it through the C ABI, twice in a row with different inputs (the scratch keeps the first call's
contents), and checks every output against the regular maxscore_index_build and against the CPU checker,
bit for bit.
It lives in a file that pytest collects last, so a run that stops at the first failure has already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


def _random_assignment(T, E, k, seed):
    g = torch.Generator().manual_seed(seed)
    scores = torch.rand(T, E, generator=g)
    return scores.topk(k, dim=1).indices.sort(dim=1).values.to(torch.int32)


def _regular(ms, idx, T, E, k, Cap):
    ctx = ms.create(ms.make_params(T, 64, E, k, capacity=Cap), DEV)
    slot_idx = torch.empty(T, k, dtype=torch.int32, device=DEV)
    slot_token = torch.empty(E, Cap, dtype=torch.int32, device=DEV)
    load = torch.empty(E, dtype=torch.int32, device=DEV)
    ms.index_build(ctx, idx, slot_idx, slot_token, load)
    torch.cuda.synchronize()
    return slot_idx.cpu().numpy(), slot_token.cpu().numpy(), load.cpu().numpy()


def test_index_build_noalloc_matches_regular_entry_point_twice(orc):
    from paper_2508_12801_b200 import binding as ms
    assert torch.cuda.is_available()
    # two calls in a row; the second is smaller, so stale scratch from the first would show
    for (T, E, k, seed) in [(5000, 64, 8, 1), (1300, 16, 2, 2)]:
        idx = _random_assignment(T, E, k, seed).to(DEV)
        Cap = int(torch.bincount(idx.flatten().cpu().long(), minlength=E).max()) + 3   # room for padding slots
        want = _regular(ms, idx, T, E, k, Cap)
        slot_idx = torch.full((T, k), -7, dtype=torch.int32, device=DEV)
        slot_token = torch.full((E, Cap), -7, dtype=torch.int32, device=DEV)
        load = torch.full((E,), -7, dtype=torch.int32, device=DEV)
        ms.index_build_noalloc(T, E, k, Cap, idx, slot_idx, slot_token, load)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(slot_idx.cpu().numpy(), want[0])
        np.testing.assert_array_equal(slot_token.cpu().numpy(), want[1])
        np.testing.assert_array_equal(load.cpu().numpy(), want[2])
        # and against the CPU checker's index build of the same assignment
        o_slot, o_tok, o_load = orc.index_build(idx.cpu().numpy(), E, Cap)
        np.testing.assert_array_equal(slot_idx.cpu().numpy(), o_slot)
        np.testing.assert_array_equal(slot_token.cpu().numpy(), o_tok)
        np.testing.assert_array_equal(load.cpu().numpy(), o_load)


def test_index_build_noalloc_rejects_sizes_beyond_its_scratch():
    from paper_2508_12801_b200 import binding as ms
    dummy = torch.zeros(16, dtype=torch.int32, device=DEV)
    for (T, E, k, want) in [((1 << 20) + 1, 8, 2, 6), (1024, 129, 2, 6), (1024, 16, 9, 6), (0, 8, 2, 1),
                            (1024, 4, 5, 2)]:
        with pytest.raises(ms.MaxScoreError) as ei:
            ms.index_build_noalloc(T, E, k, 8, dummy, dummy, dummy, dummy)
        assert ei.value.status == want
    lib = C.CDLL(ms.LIB_PATH)
    assert lib.maxscore_index_build_noalloc(8, 4, 2, 4, None, None, None, None, None) == 1

"""GPU test of mok_schedule_noalloc, the schedule entry point for callers that cannot allocate device memory (a
serving loop that must avoid cudaMalloc's device-wide synchronisation, a process whose framework owns all of HBM, a
plug-in that only receives input and output buffers).  Its scratch is a fixed array inside the library, shared by all
calls and never cleared as a whole, so the test makes two calls in a row with different sizes and checks each,
bit for bit (the outputs are integers), against mok_schedule with a caller-owned workspace and against the CPU
oracle's schedule of the same routes.  This file sorts last
on purpose: a failure here cannot hide the result of any other test under `pytest -x`."""
import numpy as np
import pytest
import torch

from oracle import mok_ref

pytestmark = pytest.mark.gpu


def test_noalloc_schedule_matches_workspace_schedule_on_consecutive_calls():
    from paper_2609_36070_b200 import mok
    gen = torch.Generator(device="cpu").manual_seed(1234)
    first = None
    for T, E, k in [(4000, 96, 8), (1111, 300, 3)]:          # second call is smaller: stale scratch must not leak
        idx = torch.randint(0, E, (T, k), generator=gen, dtype=torch.int32)
        idx[idx == 5] = 6                                     # an empty expert
        idx = idx.cuda()
        ws = mok.alloc_workspace(T, 8, 8, 0, E, k)
        want = mok.mok_schedule(idx, E, ws)
        assert mok.mok_read_status(ws) == 0
        got = mok.mok_schedule_noalloc(idx, E)
        torch.cuda.synchronize()
        for name, a, b in zip(("counts", "offsets", "perm", "inv_perm"), want, got):
            assert torch.equal(a, b), name
        ref = mok_ref.schedule(idx.cpu().numpy().ravel(), E)       # the oracle's stable counting sort of the same routes
        for name, a, b in zip(("counts", "offsets", "perm", "inv_perm"), ref, got):
            assert np.array_equal(a, b.cpu().numpy()), name
        assert int(got[0].sum()) == T * k and int(got[0][5]) == 0
        if first is None:
            first = (idx, got)
    # the first problem again, after the scratch held a different one: same bits as before
    again = mok.mok_schedule_noalloc(first[0], 96)
    torch.cuda.synchronize()
    for a, b in zip(first[1], again):
        assert torch.equal(a, b)


def test_noalloc_schedule_rejects_sizes_beyond_its_fixed_scratch():
    from paper_2609_36070_b200 import mok
    T, k, E = mok.MOK_NOALLOC_MAX_ROUTES // 8 + 1, 8, 64
    idx = torch.zeros((T, k), dtype=torch.int32, device="cuda")
    with pytest.raises(mok.MokError) as e:
        mok.mok_schedule_noalloc(idx, E)
    assert e.value.status == mok.MOK_ERR_SHAPE
    # exactly at the limit is accepted
    idx = torch.randint(0, E, (mok.MOK_NOALLOC_MAX_ROUTES // 8, 8), dtype=torch.int32).cuda()
    counts, offsets, perm, inv = mok.mok_schedule_noalloc(idx, E)
    torch.cuda.synchronize()
    assert int(offsets[-1]) == mok.MOK_NOALLOC_MAX_ROUTES

"""tt_encode_static: the entry point for callers that cannot allocate device memory (a component
inside someone else's serving process, or a latency-critical thread) must give exactly what
tt_encode gives.  Collected last on purpose (file name), so a failure here cannot hide other tests."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu


def test_static_scratch_entry_point_matches_tt_encode_twice_in_a_row():
    import torch
    import paper_2607_29678_b200 as tt
    from gpu_util import gpu_encode, gpu_vocab, to_dev

    v = gpu_vocab("C2")
    ids = torch.empty(tt.TT_STATIC_MAX_LEN, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # two different inputs back to back: the second call meets the first call's leftovers in the scratch
    for seed, n_chars in ((1, 150_000), (2, 9_000), (3, 150_000)):
        text = wl.generate(wl.KIND_MIX_UNI, seed, n_chars)
        assert text.size <= tt.TT_STATIC_MAX_LEN
        want, want_status = gpu_encode(v, text)
        assert want_status == 0
        d = to_dev(text)
        v.encode_static(d, ids, count, status, length=text.size)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = ids[:int(count.item())].cpu().numpy()
        assert got.size == want.size and np.array_equal(got, want)
    # too large: refused on the host with a clear code, nothing enqueued
    big = torch.zeros(tt.TT_STATIC_MAX_LEN + 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(tt.TokTierError) as e:
        v.encode_static(big, ids, count, status)
    assert e.value.code == tt.TT_ERR_TOO_LARGE

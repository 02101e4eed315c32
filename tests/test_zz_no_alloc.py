"""tt_encode_static: the entry point for callers that cannot allocate device memory (a component inside
someone else's serving process whose memory pool belongs to the host framework, or a latency-critical thread
that must not block in an allocation) must give exactly what tt_encode gives -- and what the oracle gives.
Collected last on purpose (file name), so a failure here cannot hide other tests."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu


def _cut_to_bytes(text, n):
    """The longest prefix of at most n bytes that ends on a character boundary."""
    n = min(n, text.size)
    while n < text.size and n > 0 and (text[n] & 0xC0) == 0x80:
        n -= 1
    return text[:n]


def test_static_scratch_entry_point_matches_tt_encode_and_the_oracle():
    import torch
    import paper_2607_29678_b200 as tt
    from gpu_util import cpu_vocab, gpu_encode, gpu_vocab, same, to_dev

    v, cv = gpu_vocab("C2"), cpu_vocab("C2")
    ids = torch.empty(tt.TT_STATIC_MAX_LEN, dtype=torch.int32, device="cuda")
    count = torch.zeros(1, dtype=torch.int64, device="cuda")
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    # different inputs back to back (each call meets the previous call's leftovers in the scratch), among them
    # one of exactly the largest accepted length and an empty one
    texts = [wl.generate(wl.KIND_MIX_UNI, 1, 150_000), wl.generate(wl.KIND_MIX_UNI, 2, 9_000),
             _cut_to_bytes(wl.generate(wl.KIND_MIX, 4, tt.TT_STATIC_MAX_LEN + 100), tt.TT_STATIC_MAX_LEN),
             np.zeros(0, dtype=np.uint8), wl.generate(wl.KIND_MIX_UNI, 3, 150_000)]
    assert texts[2].size == tt.TT_STATIC_MAX_LEN
    dev = [to_dev(t) for t in texts]
    for t, d in zip(texts, dev):
        assert t.size <= tt.TT_STATIC_MAX_LEN
        v.encode_static(d, ids, count, status, length=t.size)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        got = ids[:int(count.item())].cpu().numpy()
        want = cv.encode(t, wl.CONFIGS["C2"].pattern_id, nthreads=4)[0] if t.size else np.zeros(0, dtype=np.int32)
        assert same(got, want)
        via_workspace, ws_status = gpu_encode(v, t)
        assert ws_status == 0 and same(got, via_workspace)
    # the calls allocated no device memory: what the driver reports as free did not move (the comparison calls above
    # went through torch's caching allocator; run the static calls alone once more to be sure of the attribution)
    torch.cuda.synchronize()
    before = torch.cuda.mem_get_info()[0]
    for t, d in zip(texts, dev):
        v.encode_static(d, ids, count, status, length=t.size)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == before
    # too large: refused on the host with a clear code, nothing enqueued
    big = torch.zeros(tt.TT_STATIC_MAX_LEN + 1, dtype=torch.uint8, device="cuda")
    with pytest.raises(tt.TokTierError) as e:
        v.encode_static(big, ids, count, status)
    assert e.value.code == tt.TT_ERR_TOO_LARGE

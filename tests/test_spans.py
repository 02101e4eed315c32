"""Span export (paper App. E.3): byte and character spans of the tokens.  Oracle pins (CPU) and GPU parity."""
import numpy as np
import pytest

import oracle
import workloads as wl
from gpu_util import cpu_vocab, gpu_vocab, to_dev, same
from patterns import PATTERNS


def test_oracle_spans_hand_example():
    # merges: (a,b)->256, (é as C3 A9)->257 ; text "abéab" = 61 62 C3 A9 61 62
    merges = np.array([[97, 98, 256], [0xC3, 0xA9, 257]], dtype=np.int32)
    v = oracle.Vocab(merges)
    text = "abéab".encode()
    ids, _ = v.encode(text, 0)
    assert list(ids) == [256, 257, 256]
    b, c = v.spans(text, ids)
    assert list(b) == [0, 2, 4, 6] and list(c) == [0, 2, 3, 5]
    # a vocabulary without the é merge splits the character: the second half starts "inside" character 2
    v2 = oracle.Vocab(merges[:1])
    ids2, _ = v2.encode(text, 0)
    assert list(ids2) == [256, 0xC3, 0xA9, 256]
    b2, c2 = v2.spans(text, ids2)
    assert list(b2) == [0, 2, 3, 4, 6] and list(c2) == [0, 2, 3, 3, 5]


@pytest.mark.parametrize("name", ["C2", "C4"])
def test_oracle_spans_against_string_slicing_and_tiktoken(name):
    cfg = wl.CONFIGS[name]
    v = cpu_vocab(name)
    text = wl.request(cfg, n_chars=30_000)
    ids, _ = v.encode(text, cfg.pattern_id)
    b, c = v.spans(text, ids)
    raw = text.tobytes()
    s = raw.decode("utf-8")
    on_boundary = (text[np.minimum(b[:-1], text.size - 1)] & 0xC0) != 0x80
    for i in np.flatnonzero(on_boundary)[::37]:
        assert len(raw[:b[i]].decode("utf-8")) == c[i]
    assert c[-1] == len(s) and b[-1] == len(raw)
    tiktoken = pytest.importorskip("tiktoken")
    toks = [v.token_bytes(i) for i in range(256 + v.n_merges)]
    enc = tiktoken.Encoding("spans", pat_str=PATTERNS[cfg.pattern_id], mergeable_ranks={t: i for i, t in enumerate(toks)}, special_tokens={})
    _, offs = enc.decode_with_offsets([int(i) for i in ids])
    offs = np.asarray(offs)
    assert same(offs[on_boundary], c[:-1][on_boundary])


@pytest.mark.gpu
@pytest.mark.parametrize("name,n_chars", [("C1", None), ("C2", None), ("C3", None), ("C4", 500_000)])
def test_gpu_spans_match_oracle(name, n_chars):
    import torch
    import paper_2607_29678_b200 as tt
    cfg = wl.CONFIGS[name]
    gv, cv = gpu_vocab(name), cpu_vocab(name)
    text = wl.request(cfg, n_chars=n_chars)
    d = to_dev(text)
    bufs = gv.alloc(text.size)
    gv.encode(d, bufs, length=text.size)
    boff = torch.empty(text.size + 2, dtype=torch.int32, device="cuda")
    coff = torch.empty(text.size + 2, dtype=torch.int32, device="cuda")
    gv.spans(bufs["ids"], bufs["count"], text.size, boff, coff, bufs["status"])
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == 0
    n = int(bufs["count"].item())
    ids = bufs["ids"][:n].cpu().numpy()
    wb, wc = cv.spans(text, ids)
    assert same(boff[:n + 1].cpu().numpy(), wb)
    assert same(coff[:n + 1].cpu().numpy(), wc)
    # ids that do not belong to the text are reported, not trusted
    gv.spans(bufs["ids"], bufs["count"], text.size + 1, boff, coff, bufs["status"])
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == tt.TT_ERR_BAD_IDS
    bad = bufs["ids"].clone(); bad[0] = 10_000_000
    gv.spans(bad, bufs["count"], text.size, boff, coff, bufs["status"])
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == tt.TT_ERR_BAD_IDS
    # empty input
    zero = torch.zeros(1, dtype=torch.int64, device="cuda")
    gv.spans(bufs["ids"], zero, 0, boff, coff, bufs["status"])
    torch.cuda.synchronize()
    assert int(bufs["status"].item()) == 0 and int(boff[0].item()) == 0 and int(coff[0].item()) == 0

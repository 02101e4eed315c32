"""Shadow verifier (paper Sec. 4.4) -- host only, runs without a GPU: sampled re-tokenization by a reference
engine on a background thread, exact id comparison, quarantine with a content hash, visible drop counter."""
import time

import numpy as np

import oracle
import workloads as wl
import paper_2607_29678_b200 as tt


def _fnv1a64(data: bytes) -> int:
    h = 0xCBF29CE484222325
    for b in data:
        h = ((h ^ b) * 0x100000001B3) & 0xFFFFFFFFFFFFFFFF
    return h


def _vocab():
    cfg = wl.CONFIGS["C1"]
    merges, byte_map = wl.load_vocab(cfg)
    return oracle.Vocab(merges, byte_map), cfg.pattern_id


def test_full_rate_catches_and_quarantines_a_wrong_sequence():
    v, pat = _vocab()
    ver = tt.Verifier(lambda text: v.encode(text, pat)[0], sample_rate=1.0, queue_cap=256)
    texts = [wl.generate(wl.KIND_MIX, 10 + k, 300).tobytes() for k in range(20)]
    for k, t in enumerate(texts):
        ids = v.encode(t, pat)[0].copy()
        if k == 7:
            ids[5] += 1                      # a wrong id
        if k == 13:
            ids = ids[:-2]                   # a short sequence
        assert ver.submit(t, ids) == 1
    ver.drain()
    st = ver.stats()
    assert st == {"submitted": 20, "sampled": 20, "checked": 20, "mismatches": 2, "dropped": 0}
    q = sorted(ver.quarantined(i) for i in range(2))
    want = sorted([(_fnv1a64(texts[7]), len(texts[7]), 5),
                   (_fnv1a64(texts[13]), len(texts[13]), len(v.encode(texts[13], pat)[0]) - 2)])
    assert q == want
    ver.close()


def test_sampling_rate_and_determinism():
    v, pat = _vocab()
    t = b"hello world"
    ids = v.encode(t, pat)[0]
    picks = []
    for _ in range(2):
        ver = tt.Verifier(lambda text: v.encode(text, pat)[0], sample_rate=0.05, queue_cap=100000, seed=42)
        picks.append([ver.submit(t, ids) for _ in range(4000)])
        ver.drain()
        st = ver.stats()
        assert st["submitted"] == 4000 and st["checked"] == st["sampled"] and st["mismatches"] == 0
        assert 120 <= st["sampled"] <= 290            # 5 % of 4,000 = 200, binomial sd about 14
        ver.close()
    assert picks[0] == picks[1]                        # the seed fixes which submissions are sampled


def test_falling_behind_drops_samples_and_counts_them():
    v, pat = _vocab()

    def slow(text):
        time.sleep(0.02)
        return v.encode(text, pat)[0]
    ver = tt.Verifier(slow, sample_rate=1.0, queue_cap=2)
    t = b"some text to check"
    ids = v.encode(t, pat)[0]
    t0 = time.perf_counter()
    results = [ver.submit(t, ids) for _ in range(40)]
    assert time.perf_counter() - t0 < 0.5              # submit never waits for the reference engine
    ver.drain()
    st = ver.stats()
    assert st["dropped"] == results.count(2) > 0
    assert st["checked"] == results.count(1) and st["checked"] + st["dropped"] == 40 and st["mismatches"] == 0
    ver.close()


def test_reference_failure_counts_as_mismatch():
    def broken(text):
        raise RuntimeError("engine down")
    ver = tt.Verifier(broken, sample_rate=1.0)
    ver.submit(b"abc", np.array([1, 2, 3], dtype=np.int32))
    ver.drain()
    assert ver.stats()["mismatches"] == 1 and ver.quarantined(0)[2] == -2
    ver.close()

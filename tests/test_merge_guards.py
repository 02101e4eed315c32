"""Host logic of the merge rounds (no GPU): the guards that let a round merge more than the lowest rank.

Paper Sec. 4.2 fixes the result of BPE on a piece as that of the sequential algorithm (always the leftmost pair of
the lowest rank).  The kernels merge, in one round, every pair (x, y) of rank r whose left neighbour u and right
neighbour w satisfy r < cl(u, x) and r <= cr(y, w), plus the pairs of the round's lowest rank, plus every other
pair of a run of identical pairs behind such a pair.  Checked here:
  * the (rank, cl, cr) triples the library builds on the host against their definition, by brute force over the
    merge trees of a small vocabulary;
  * a plain Python model of the rounds that takes its triples from the library, against the oracle's sequential
    BPE, on random pieces over several alphabets and on the stored vocabularies.
"""
import random

import numpy as np
import pytest

import oracle
import workloads as wl

INF = 1 << 40


def _tt():
    import paper_2607_29678_b200 as tt
    return tt


def _small_vocab(seed, n_merges=300, alphabet=b"abcd \t"):
    """A random merge list over a small alphabet (every operand defined before use, no duplicate pair)."""
    rng = random.Random(seed)
    toks = list(alphabet)
    seen, merges = set(), []
    while len(merges) < n_merges:
        a, b = rng.choice(toks), rng.choice(toks)
        if (a, b) in seen:
            continue
        seen.add((a, b))
        merges.append((a, b, 256 + len(merges)))
        toks.append(256 + len(merges) - 1)
    return np.array(merges, dtype=np.int32)


def _brute_guards(merges):
    """cl / cr straight from the definition: spines of the merge trees."""
    left = {int(c): int(a) for a, b, c in merges}
    right = {int(c): int(b) for a, b, c in merges}

    def spine(t, child):
        out = [t]
        while t in child:
            t = child[t]
            out.append(t)
        return out

    rank, cl, cr = {}, {}, {}
    for r, (a, b, c) in enumerate(merges.tolist()):
        rank[(a, b)] = r
        for u in spine(a, right):
            cl[(u, b)] = min(cl.get((u, b), INF), r)
        for w in spine(b, left):
            cr[(a, w)] = min(cr.get((a, w), INF), r)
    return rank, cl, cr


def test_guard_triples_match_their_definition():
    tt = _tt()
    merges = _small_vocab(1)
    rank, cl, cr = _brute_guards(merges)
    ids = sorted(set(merges[:, 2].tolist()) | set(b"abcd \t") | {ord("z")})
    L, R = np.meshgrid(ids, ids, indexing="ij")
    got = tt.pair_info_host(merges, None, L.ravel(), R.ravel())
    for (a, b), (r, x, y) in zip(zip(L.ravel().tolist(), R.ravel().tolist()), got.tolist()):
        assert r == rank.get((a, b), -1) and x == (cl.get((a, b), -1)) and y == (cr.get((a, b), -1)), (a, b)
    assert (got[:, 1] >= 0).sum() > (got[:, 0] >= 0).sum()          # guards exist for pairs that are no merge


def _round_step(toks, tri):
    """One round of the kernels' schedule: tri[i] = (rank, cl, cr) of the pair (toks[i], toks[i + 1]), INF for
    none.  Returns the new token list, or None at the fixpoint."""
    m = len(toks)
    r = [t[0] for t in tri]
    if not r or min(r) >= INF:
        return None
    mn = min(r)
    sel = [False] * (m - 1)
    head_ok, head = False, 0
    for i in range(m - 1):
        same_as_left = i >= 1 and r[i] < INF and toks[i - 1] == toks[i] == toks[i + 1]
        if not same_as_left:
            head = i
            head_ok = r[i] < INF and (r[i] == mn or i == 0 or r[i] < tri[i - 1][1])
        right_ok = r[i] == mn or i == m - 2 or r[i] <= tri[i + 1][2]
        sel[i] = r[i] < INF and head_ok and (i - head) % 2 == 0 and right_ok
    assert not any(sel[i] and sel[i + 1] for i in range(m - 2))
    assert any(sel)
    out, i = [], 0
    while i < m:
        if i < m - 1 and sel[i]:
            out.append(256 + r[i])
            i += 2
        else:
            out.append(toks[i])
            i += 1
    return out


def _rounds_many(pieces, batch_info):
    """All pieces in lock step, one batched triple query per round.  Returns (token lists, rounds per piece)."""
    state = [list(p) for p in pieces]
    rounds = [0] * len(state)
    live = [k for k, t in enumerate(state) if len(t) > 1]
    cache = {}
    while live:
        need = sorted({pr for k in live for pr in zip(state[k][:-1], state[k][1:])} - cache.keys())
        if need:
            for pr, t in zip(need, batch_info(need)):
                cache[pr] = tuple(INF if x < 0 else x for x in t)
        nxt = []
        for k in live:
            toks = state[k]
            out = _round_step(toks, [cache[pr] for pr in zip(toks[:-1], toks[1:])])
            if out is not None:
                state[k] = out
                rounds[k] += 1
                if len(out) > 1:
                    nxt.append(k)
        live = nxt
    return state, rounds


@pytest.mark.parametrize("seed", [2, 3, 4])
def test_round_model_equals_sequential_bpe_small_vocab(seed):
    tt = _tt()
    alphabet = b"ab \t" if seed == 2 else b"abcdefg"
    merges = _small_vocab(seed, n_merges=400, alphabet=alphabet)
    ov = oracle.Vocab(merges, None)
    rng = random.Random(seed)
    pieces = []
    for trial in range(300):
        n = rng.choice([1, 2, 3, 5, 8, 13, 31, 32, 33, 64, 200, 700])
        pieces.append(bytes(rng.choice(alphabet) for _ in range(n)) if trial % 5 else bytes([rng.choice(alphabet)]) * n)
    got, rounds = _rounds_many(pieces, lambda prs: tt.pair_info_host(merges, None, [p[0] for p in prs], [p[1] for p in prs]).tolist())
    fewer = 0
    for piece, toks, nr in zip(pieces, got, rounds):
        want = ov.bpe(np.frombuffer(piece, dtype=np.uint8)).tolist()
        assert toks == want, piece
        fewer += nr < len(piece) - len(want)
    assert fewer > 100          # the guards do merge several ranks per round


@pytest.mark.parametrize("name", ["C1", "C3"])
def test_round_model_equals_sequential_bpe_stored_vocab(name):
    tt = _tt()
    cfg = wl.CONFIGS[name]
    merges, byte_map = wl.load_vocab(cfg)
    ov = oracle.Vocab(merges, byte_map)
    text = wl.request(cfg, n_chars=min(cfg.n_chars, 60_000))
    starts = np.append(oracle.pretokenize(text, cfg.pattern_id), text.size)
    pieces = sorted({text[a:b].tobytes() for a, b in zip(starts[:-1], starts[1:]) if b - a >= 6}, key=len, reverse=True)[:150]
    rng = random.Random(5)
    pieces += [bytes(rng.choice(b"abcdefghijklmnopqrstuvwxyz") for _ in range(n)) for n in (20, 48, 120, 400)]
    pieces += [bytes(rng.choice(b" \t") for _ in range(300)), b" " * 257, b"ab" * 100]
    got, rounds = _rounds_many(pieces, lambda prs: tt.pair_info_host(merges, byte_map, [p[0] for p in prs], [p[1] for p in prs]).tolist())
    for piece, toks in zip(pieces, got):
        assert toks == ov.bpe(np.frombuffer(piece, dtype=np.uint8)).tolist(), piece
    assert max(rounds) < 40

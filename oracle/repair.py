"""Incremental repair on append (paper Sec. 3.3) -- TEST INFRASTRUCTURE ONLY, like the rest of ``oracle/``.

A session holds the tokenization of a text A as records (byte position, id).  For a request A + B the last
``w`` characters of A (512 by default) plus B are tokenized afresh; the longest run of records on which the
cached and the fresh sequence agree in position and id is looked for inside the old part of the window; the
*stable boundary check* admits the run if (1) it has at least two tokens, (2) it covers more characters than
the longest token of the vocabulary and (3) it contains a stable boundary: a character-class transition at
which the pieces to the right do not depend on the text to the left.  Then cached records are kept up to the
end of the run and fresh ones after it.  Otherwise w doubles, at most five times, and after that the whole
text is tokenized.

Readings where the paper leaves a choice (the same are taken by the CUDA session, which shares no code with
this file):
  * among several longest runs the rightmost is taken;
  * the window is the last w characters of A; a window that reaches the start of A is a full tokenization;
  * stable boundaries (both pattern lineages; a subset of the positions that always begin a piece, chosen so
    that one rule serves all patterns): at a character c preceded by a character q of the same document,
      - c is whitespace and q is a letter or a number;
      - c is a number and q is not a number;
      - c is a letter and q is a number;
      - c is neither letter, number, whitespace nor mark, is not an apostrophe, and q is a letter or a number;
    the boundary must be the start of one of the run's tokens.

Everything here is plain Python over the oracle's encode; it is slow and meant for small cases.
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np

from . import K_LB, K_LL, K_LU, K_M, K_N, K_O, K_W, Vocab, class_table

DEFAULT_WINDOW = 512
MAX_WIDENINGS = 5


def _char_at(text: bytes, p: int):
    """(code point, length) of the character that starts at byte p of valid UTF-8."""
    b = text[p]
    n = 1 if b < 0x80 else 2 if b < 0xE0 else 3 if b < 0xF0 else 4
    return ord(text[p:p + n].decode("utf-8")), n


def _prev_start(text: bytes, p: int) -> int:
    q = p - 1
    while q > 0 and (text[q] & 0xC0) == 0x80:
        q -= 1
    return q


def is_stable_boundary(text: bytes, p: int) -> bool:
    """Is byte position p (a character start, 0 < p < len) a stable boundary in the sense above?"""
    if p <= 0 or p >= len(text) or (text[p] & 0xC0) == 0x80:
        return False
    tab = class_table()
    cp, _ = _char_at(text, p)
    cq, _ = _char_at(text, _prev_start(text, p))
    c, q = int(tab[cp]), int(tab[cq])
    letter = (K_LL, K_LU, K_LB)
    q_ln = q in letter or q == K_N
    if c == K_W:
        return q_ln
    if c == K_N:
        return q != K_N
    if c in letter:
        return q == K_N
    if c == K_O:
        return cp != 0x27 and q_ln
    return False          # marks


def max_token_chars(vocab: Vocab) -> int:
    """Characters (non-continuation bytes) of the longest entry of the vocabulary."""
    best = 1
    for r in vocab.merges[:, 2].tolist():
        s = vocab.token_bytes(int(r))
        best = max(best, sum((b & 0xC0) != 0x80 for b in s))
    return best


@dataclass
class Session:
    vocab: Vocab
    pattern: int
    window: int = DEFAULT_WINDOW
    text: bytes = b""
    ids: list = field(default_factory=list)
    off: list = field(default_factory=lambda: [0])       # off[i] = byte start of token i, off[-1] = len(text)
    _maxtok: int = 0

    def __post_init__(self):
        self._maxtok = max_token_chars(self.vocab)

    def _encode(self, data: bytes):
        ids, _ = self.vocab.encode(data, self.pattern)
        byte_off, char_off = self.vocab.spans(data, ids) if len(data) else (np.zeros(1, np.int64), np.zeros(1, np.int64))
        return ids.tolist(), byte_off.tolist(), char_off.tolist()

    def _window_start(self, w: int) -> int:
        """Byte offset of the character that lies w characters before the end of the stored text (0 if fewer)."""
        p, left = len(self.text), w
        while p > 0 and left > 0:
            p = _prev_start(self.text, p)
            left -= 1
        return p

    def append(self, more: bytes, check_boundary: bool = True) -> dict:
        """Appends `more`; returns what happened.  check_boundary=False drops condition (3) -- only for the test
        that shows why the condition is needed."""
        old_len = len(self.text)
        full = self.text + more
        info = {"attempts": 0, "window_chars": 0, "window_start": 0, "run_tokens": 0, "splice_byte": 0}
        w = self.window
        for attempt in range(MAX_WIDENINGS + 1):
            ws = self._window_start(w)
            info["attempts"] = attempt + 1
            if ws == 0:
                break                                       # the window is the whole text
            fids, foff, fchar = self._encode(full[ws:])
            # fresh records that lie in the old part, matched against the cached records by position and id
            cached_at = {self.off[i]: i for i in range(len(self.ids))}
            eq = []
            for j in range(len(fids)):
                p, e = ws + foff[j], ws + foff[j + 1]
                i = cached_at.get(p)
                eq.append(e <= old_len and i is not None and self.ids[i] == fids[j] and self.off[i + 1] == e)
            # longest run of agreement, the rightmost among equals
            best = (0, 0)
            j = 0
            while j < len(eq):
                if not eq[j]:
                    j += 1
                    continue
                k = j
                while k < len(eq) and eq[k]:
                    k += 1
                if k - j >= best[1] - best[0]:
                    best = (j, k)
                j = k
            j0, j1 = best
            ok = j1 - j0 >= 2 and fchar[j1] - fchar[j0] > self._maxtok
            if ok and check_boundary:
                ok = any(is_stable_boundary(full, ws + foff[j]) for j in range(j0, j1))
            if ok:
                i1 = cached_at[ws + foff[j1 - 1]] + 1
                self.ids = self.ids[:i1] + fids[j1:]
                self.off = self.off[:i1] + [ws + x for x in foff[j1:]]
                self.text = full
                info.update(window_chars=w, window_start=ws, run_tokens=j1 - j0, splice_byte=ws + foff[j1])
                return info
            w *= 2
        ids, off, _ = self._encode(full)
        self.ids, self.off, self.text = ids, off, full
        info.update(window_chars=0, window_start=0, run_tokens=0, splice_byte=0)
        return info

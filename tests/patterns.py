"""Test-side statement of the two pre-tokenization patterns as regular expressions for a
backtracking engine (the third-party ``regex`` module).  The oracle itself never uses a regex
engine; these strings exist only to pin it."""
CON = r"'(?:[sStTmMdD]|[rR][eE]|[vV][eE]|[lL][lL])"
P0 = (CON
      + r"|[^\r\n\p{L}\p{N}]?\p{L}+"
      + r"|\p{N}{1,3}"
      + r"| ?[^\s\p{L}\p{N}]+[\r\n]*"
      + r"|\s*[\r\n]+"
      + r"|\s+(?!\S)"
      + r"|\s+")
U = r"[\p{Lu}\p{Lt}\p{Lm}\p{Lo}\p{M}]"
LW = r"[\p{Ll}\p{Lm}\p{Lo}\p{M}]"
P1 = (r"[^\r\n\p{L}\p{N}]?" + U + "*" + LW + "+" + "(?:" + CON + ")?"
      + r"|[^\r\n\p{L}\p{N}]?" + U + "+" + LW + "*" + "(?:" + CON + ")?"
      + r"|\p{N}{1,3}"
      + r"| ?[^\s\p{L}\p{N}]+[\r\n/]*"
      + r"|\s*[\r\n]+"
      + r"|\s+(?!\S)"
      + r"|\s+")
# pattern 2: pattern 0 with single-digit number pieces (the paper's family table lists a "\\p{N} single" front end)
P2 = P0.replace(r"|\p{N}{1,3}", r"|\p{N}")
assert P2 != P0
PATTERNS = [P0, P1, P2]


def engine_starts(compiled, s: str):
    """Successive leftmost-first matches from position 0; returns piece start BYTE offsets."""
    out, p, b = [], 0, 0
    while p < len(s):
        m = compiled.match(s, p)
        assert m and m.end() > p
        out.append(b)
        b += len(s[p:m.end()].encode("utf-8"))
        p = m.end()
    return out


# pattern 3: three splitters in sequence, matches isolated, unmatched spans kept as pieces (paper Sec. 4.1)
SPLIT3_A = r"\p{N}{1,3}"
SPLIT3_B = r"[\p{Lm}\p{Lo}]+"


def split_isolated(compiled, s: str, lo: int, hi: int):
    """Spans of s[lo:hi]: the matches of `compiled` and the gaps between them, in order."""
    out, p = [], lo
    for m in compiled.finditer(s, lo, hi):
        if m.start() > p:
            out.append((p, m.start()))
        out.append((m.start(), m.end()))
        p = m.end()
    if p < hi:
        out.append((p, hi))
    return out


def engine_starts_split3(ra, rb, r0, s: str):
    """Piece start BYTE offsets of the composition A, B, then pattern 0 on every piece as a text of its own."""
    starts = []
    for a0, a1 in split_isolated(ra, s, 0, len(s)):
        for b0, b1 in split_isolated(rb, s, a0, a1):
            piece = s[b0:b1]
            base = len(s[:b0].encode("utf-8"))
            starts.extend(base + x for x in engine_starts(r0, piece))
    return starts

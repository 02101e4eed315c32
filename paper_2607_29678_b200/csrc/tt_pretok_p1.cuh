// Pattern 1 (o200k-style) piece-start predicate.
//
// Paper Sec. 4.1: this lineage adds a case-boundary rule and a sparse contraction path to the
// run-local rules, and Unicode marks take a narrow sparse fallback while the common path stays
// vectorised.  Here the vectorised path covers number runs, whitespace runs, punctuation runs with
// their [\r\n/]* tails, word starts with the one-character prefix, the lower->upper case boundary and
// the contraction suffix after a word.  Three constructs are not decided by those rules: a mark, an
// upper-case letter that follows a caseless letter, and an apostrophe between letters that has another
// apostrophe two or three bytes before it (a chain of possible contraction suffixes).  The second
// kind is decided from the tile's class masks wherever they reach (tt_resolve_upper_after_caseless).
// What stays unresolved marks the text from the last *sure* piece start before it up to the next sure
// piece start; a thread whose chunk contains such bytes re-derives them by matching sequentially from
// that sure start (matching from a piece start never looks behind it).  Sure starts are positions that
// begin a piece whatever surrounds them: a document start, the first digit of a number run, whitespace
// or punctuation right after a digit, whitespace or non-apostrophe punctuation right after a letter, a
// letter right after a digit or a CR/LF, a one-byte blank right before a letter, a letter after two
// punctuation characters, and the decided case boundaries.
#pragma once
#include "tt_pretok.cuh"

struct SeqCtx {                 // what the sequential matcher needs to read the text itself
    const u8* base;
    long long lo, hi;
    const u32* docmask;         // or null: one document
    ClassTables T;
    mutable long long reach;    // highest text position (exclusive) a match has examined so far
};

// ---- sequential matcher over the raw text (sparse path) ---------------------------------------------
struct SeqChar { u32 cls; u32 byte; int len; };   // byte = the ASCII byte, or 0x100 for multi-byte characters

TT_HD SeqChar tt_seq_char(const SeqCtx& C, long long g, long long end) {
    SeqChar r;
    u32 b = C.base[g];
    if (b < 0x80) { r.cls = C.T.ascii[b] & 7; r.byte = b; r.len = 1; if (g + 1 > C.reach) C.reach = g + 1; return r; }
    int n = b >= 0xF0 ? 4 : b >= 0xE0 ? 3 : 2;
    if (g + n > end) n = (int)(end - g);
    if (g + n > C.reach) C.reach = g + n;
    u32 cp = b & (0x7Fu >> (b >= 0xF0 ? 4 : b >= 0xE0 ? 3 : 2));
    for (int k = 1; k < n; k++) cp = (cp << 6) | (C.base[g + k] & 0x3F);
    if (cp > 0x10FFFF) cp = 0xFFFD;                  // malformed input: the result is discarded anyway
    r.cls = tt_class_of(cp, C.T); r.byte = 0x100; r.len = n < 1 ? 1 : n;
    return r;
}
TT_HD bool tt_cls_word(u32 c) { return c == CC_LOWER || c == CC_UPPER || c == CC_CASELESS || c == CC_MARK; }
TT_HD bool tt_cls_up(u32 c) { return c == CC_UPPER || c == CC_CASELESS || c == CC_MARK; }      // U
TT_HD bool tt_cls_lw(u32 c) { return c == CC_LOWER || c == CC_CASELESS || c == CC_MARK; }      // Lw
TT_HD bool tt_cls_letter(u32 c) { return c == CC_LOWER || c == CC_UPPER || c == CC_CASELESS; }
TT_HD bool tt_cls_punct(u32 c) { return c == CC_OTHER || c == CC_MARK; }                        // [^\s\p{L}\p{N}]

// U* Lw+ from q (greedy U*, giving characters back until Lw+ can start); returns the end or q.
TT_HD long long tt_seq_body_lower(const SeqCtx& C, long long q, long long end) {
    long long t = q, last_lw_end = -1;
    while (t < end) {
        SeqChar ch = tt_seq_char(C, t, end);
        if (!tt_cls_word(ch.cls) || !tt_cls_up(ch.cls)) break;
        if (tt_cls_lw(ch.cls)) last_lw_end = t + ch.len;
        t += ch.len;
    }
    if (t < end) {
        SeqChar ch = tt_seq_char(C, t, end);
        if (tt_cls_word(ch.cls) && tt_cls_lw(ch.cls)) {
            long long v = t;
            while (v < end) { SeqChar c2 = tt_seq_char(C, v, end); if (!tt_cls_word(c2.cls) || !tt_cls_lw(c2.cls)) break; v += c2.len; }
            return v;
        }
    }
    return last_lw_end >= 0 ? last_lw_end : q;
}
// U+ Lw* from q
TT_HD long long tt_seq_body_upper(const SeqCtx& C, long long q, long long end) {
    long long t = q;
    while (t < end) { SeqChar ch = tt_seq_char(C, t, end); if (!tt_cls_word(ch.cls) || !tt_cls_up(ch.cls)) break; t += ch.len; }
    if (t == q) return q;
    while (t < end) { SeqChar ch = tt_seq_char(C, t, end); if (!tt_cls_word(ch.cls) || !tt_cls_lw(ch.cls)) break; t += ch.len; }
    return t;
}
// One leftmost-first match of pattern 1 at p (p < end); returns the end of the piece.
TT_HD long long tt_seq_match_p1(const SeqCtx& C, long long p, long long end) {
    const SeqChar c0 = tt_seq_char(C, p, end);
    const bool nl0 = c0.byte == '\n' || c0.byte == '\r';
    const bool prefix_ok = !nl0 && !tt_cls_letter(c0.cls) && c0.cls != CC_NUMBER;
    long long e = -1;
    for (int alt = 0; alt < 2 && e < 0; alt++) {
        if (prefix_ok && p + c0.len < end) {
            long long q = p + c0.len, v = alt == 0 ? tt_seq_body_lower(C, q, end) : tt_seq_body_upper(C, q, end);
            if (v > q) { e = v; break; }
        }
        long long v = alt == 0 ? tt_seq_body_lower(C, p, end) : tt_seq_body_upper(C, p, end);
        if (v > p) e = v;
    }
    if (e >= 0) {
        if (e + 3 > end) C.reach = end;
        if (e < end && C.base[e] == '\'') {
            u32 b1 = e + 1 < end ? C.base[e + 1] : 0, b2 = e + 2 < end ? C.base[e + 2] : 0;
            e += tt_contraction_len(b1, b2);
        }
        return e;
    }
    if (c0.cls == CC_NUMBER) {
        long long t = p; int k = 0;
        while (t < end && k < 3) { SeqChar ch = tt_seq_char(C, t, end); if (ch.cls != CC_NUMBER) break; t += ch.len; k++; }
        return t;
    }
    long long q = -1;
    if (c0.byte == ' ' && p + 1 < end && tt_cls_punct(tt_seq_char(C, p + 1, end).cls)) q = p + 1;
    else if (tt_cls_punct(c0.cls)) q = p;
    if (q >= 0) {
        while (q < end) { SeqChar ch = tt_seq_char(C, q, end); if (!tt_cls_punct(ch.cls)) break; q += ch.len; }
        while (q < end) { u32 b = C.base[q]; if (b != '\n' && b != '\r' && b != '/') break; q++; }
        if (q + 1 > C.reach) C.reach = q + 1 < end ? q + 1 : end;
        return q;
    }
    // whitespace: \s*[\r\n]+ | \s+(?!\S) | \s+
    long long t = p, last_nl_end = -1, last_char = p; int n = 0;
    while (t < end) {
        SeqChar ch = tt_seq_char(C, t, end);
        if (ch.cls != CC_SPACE) break;
        if (ch.byte == '\n' || ch.byte == '\r') last_nl_end = t + 1;
        last_char = t; t += ch.len; n++;
    }
    if (last_nl_end >= 0) return last_nl_end;
    if (t >= end) return t;
    if (n >= 2) return last_char;
    return t > p ? t : p + c0.len;
}

// First document start in [g, lim), or lim when there is none.
TT_HD long long tt_next_doc_start(const u32* docmask, long long g, long long lim) {
    while (g < lim) {
        const u32 w = docmask[g >> 5] >> (g & 31);
        if (w) { g += tt_lobit(w); break; }
        g = ((g >> 5) + 1) << 5;
    }
    return g < lim ? g : lim;
}

// Piece starts inside [g0, g0+16) obtained by matching sequentially from the piece start `from`
// (from <= g0 + 15).  Returns a 16-bit mask; bits below `from` are not produced.  The end of the
// document that contains `from` is looked up only as far as the matches look: the search begins with a
// provisional end a little past the chunk, and a match that examined the provisional end is repeated
// with the end moved out geometrically (documents can be megabytes long; pieces rarely are).
// doc_end returns an end that is exact whenever it is below g0 + 16.
TT_HD_COLD u32 tt_seq_starts_p1(const SeqCtx& C, long long from, long long g0, long long& doc_end) {
    long long end = C.hi;
    bool exact = true;
    if (C.docmask) {
        long long cap = g0 + TT_CHUNK + 64;
        if (cap > C.hi) cap = C.hi;
        end = tt_next_doc_start(C.docmask, from + 1, cap);
        exact = end < cap || cap == C.hi;
    }
    u32 bits = 0;
    long long p = from;
    for (;;) {
        const long long stop = g0 + TT_CHUNK < end ? g0 + TT_CHUNK : end;
        if (p >= stop) break;
        C.reach = 0;
        const long long e = tt_seq_match_p1(C, p, end);
        if (!exact && C.reach >= end) {                // looked at the provisional end: move it out, match again
            long long cap = end + 4 * (end - from);
            if (cap > C.hi) cap = C.hi;
            const long long ne = tt_next_doc_start(C.docmask, end, cap);
            exact = ne < cap || cap == C.hi;
            end = ne;
            continue;
        }
        if (p >= g0) bits |= 1u << (int)(p - g0);
        p = e > p ? e : p + 1;
    }
    doc_end = end;
    return bits;
}

// ---- marks inside words -------------------------------------------------------------------------------
// In pattern 1 a mark belongs to both word classes, exactly like a caseless letter, and a word match that has taken a
// letter always goes on over a mark that follows it.  So a run of marks right behind a letter lies inside that
// letter's word and behaves as caseless letters do; only a mark at the head of a run of word characters (after
// whitespace, punctuation, a digit, the start of the text) can also be punctuation and stays an unresolved construct.
// One exception: a letter that may end a contraction suffix (an apostrophe one or two bytes before it) ends its piece,
// so marks behind it are left unresolved as well.  Returns the bits of slot s (s >= 0) whose marks lie inside a word;
// the masks of the two slots before it give the look-back (a run of marks that reaches back beyond them stays
// unresolved).
TT_HD u32 tt_marks_inside_words(const u16 (*sm)[TT_SLOTS], int s) {
    const u32 own = sm[F_MARK][s];
    if (own == 0) return 0;
#define W3(f) ((s >= 2 ? (u64)sm[f][s - 2] : 0ull) | (s >= 1 ? (u64)sm[f][s - 1] << 16 : 0ull) | ((u64)sm[f][s] << 32))
    const u64 D = W3(F_DOC), Mk = W3(F_MARK) & ~D;                 // a mark that starts a document heads a run
    const u64 Lr = W3(F_LOW) | W3(F_UPP) | W3(F_CLESS), AP = W3(F_AP);
#undef W3
    const u64 starts = Mk & ~(Mk << 1);
    const u64 good = starts & (Lr << 1) & ~D & ~((AP << 2) | (AP << 3));
    const u64 inside = Mk & ~(Mk + good);                          // the carry runs through every run that starts well
    return (u32)(inside >> 32) & 0xFFFFu;
}

// ---- masks of sure piece starts and of unresolved constructs for one chunk ---------------------------
struct ChunkDoc { ChunkMasks m; u32 doc; };

TT_HD ChunkDoc tt_load_slot(const u16 (*sm)[TT_SLOTS], int s) {
    ChunkDoc c;
    c.m.lead = sm[F_LEAD][s]; c.m.oth = sm[F_OTH][s]; c.m.mark = sm[F_MARK][s]; c.m.spc = sm[F_SPC][s]; c.m.num = sm[F_NUM][s];
    c.m.low = sm[F_LOW][s]; c.m.upp = sm[F_UPP][s]; c.m.cless = sm[F_CLESS][s]; c.m.nl = sm[F_NL][s]; c.m.sp = sm[F_SP][s];
    c.m.ap = sm[F_AP][s]; c.m.sl = sm[F_SL][s]; c.m.bad = 0; c.doc = sm[F_DOC][s];
    return c;
}
// The same for three neighbouring chunks held in registers (the cooperative walks over the text): marks inside words
// become caseless letters in all three, as far as the 48 bytes show it.
TT_HD void tt_marks_inside_words_cm(ChunkDoc& p, ChunkDoc& c, ChunkDoc& n) {
    if ((p.m.mark | c.m.mark | n.m.mark) == 0) return;
#define W3(x) ((u64)p.x | ((u64)c.x << 16) | ((u64)n.x << 32))
    const u64 D = W3(doc), Mk = W3(m.mark) & ~D;
    const u64 Lr = W3(m.low) | W3(m.upp) | W3(m.cless), AP = W3(m.ap);
#undef W3
    const u64 starts = Mk & ~(Mk << 1);
    const u64 good = starts & (Lr << 1) & ~D & ~((AP << 2) | (AP << 3));
    const u64 inside = Mk & ~(Mk + good);
    const u16 ip = (u16)inside, ic = (u16)(inside >> 16), in = (u16)(inside >> 32);
    p.m.mark &= (u16)~ip; p.m.cless |= ip; c.m.mark &= (u16)~ic; c.m.cless |= ic; n.m.mark &= (u16)~in; n.m.cless |= in;
}

// p = previous chunk, c = the chunk, n = next chunk
// upcl: the unresolved constructs of the second kind (upper-case letter after a caseless letter), a subset of hard
// apch: the unresolved constructs of the third kind (apostrophe between letters with another apostrophe two or three
// bytes before it), a subset of hard
TT_HD void tt_sure_hard_cm(const ChunkDoc& p, const ChunkDoc& c, const ChunkDoc& n, u32& sure, u32& hard, u32& upcl, u32& apch) {
    // 20-bit frame: bits 0..2 = last three bytes of the previous chunk, bits 3..18 = the chunk, bit 19 = first byte of the next
#define FR(x) ((((u32)p.x) >> 13) | (((u32)c.x) << 3) | ((((u32)n.x) & 1u) << 19))
    const u32 lead = FR(m.lead), D = FR(doc);
    const u32 Lr = FR(m.low) | FR(m.upp) | FR(m.cless), N = FR(m.num), W = FR(m.spc), O = FR(m.oth), AP = FR(m.ap);
    const u32 nD = ~D;
    const u32 pLr = (Lr << 1) & nD, pN = (N << 1) & nD, pNL = (FR(m.nl) << 1) & nD, pCl = (FR(m.cless) << 1) & nD;
    const u32 nLr = (Lr >> 1) & ~(D >> 1);
    // a one-byte blank right before a letter is the letter's prefix whatever precedes it; a letter after two
    // punctuation characters (the nearer one a single byte, the farther one no slash, which a tail could have
    // taken) follows a punctuation piece that ends there
    const u32 blank_pfx = W & ~FR(m.nl) & lead & (lead >> 1) & (Lr >> 1) & ~(D >> 1);
    const u32 after_oo = Lr & ((O & lead) << 1) & ((O & ~FR(m.sl)) << 2) & nD & ~(D << 1);
    const u32 cs = D | (N & ~pN) | (W & (pLr | pN)) | (O & (pN | (~AP & pLr))) | (Lr & (pN | pNL)) | blank_pfx | after_oo;
    // an apostrophe between letters is a possible contraction suffix; it is decided locally unless another
    // apostrophe two or three bytes before it may have consumed the letter in front of it
    const u32 h2 = FR(m.upp) & pCl;
    const u32 h3 = AP & pLr & nLr & ((AP << 2) | (AP << 3));
    const u32 h = FR(m.mark) | h2 | h3;
#undef FR
    sure = ((cs & lead) >> 3) & 0xFFFFu;
    hard = ((h & lead) >> 3) & 0xFFFFu;
    upcl = ((h2 & lead) >> 3) & 0xFFFFu;
    apch = ((h3 & lead) >> 3) & 0xFFFFu;
}
TT_HD void tt_sure_hard_cm(const ChunkDoc& p, const ChunkDoc& c, const ChunkDoc& n, u32& sure, u32& hard) {
    u32 upcl, apch;
    tt_sure_hard_cm(p, c, n, sure, hard, upcl, apch);
}

// An upper-case letter (bit i of slot s) that follows a caseless letter, decided from the class masks of
// the tile: 1 = it starts a piece, 0 = it does not, -1 = left to the sparse path.
//   Going left over the caseless letters: a lower-case letter means the letters in between continue its
//   lower-case stretch, which stops at the upper-case letter, so that one starts a piece (unless the
//   lower-case letter may belong to a contraction suffix, which begins a word body of its own).  An
//   upper-case letter, a non-letter or a document start means the word body has held no lower-case
//   letter so far; its leading stretch then runs to the first lower-case letter or to the end of the
//   letter run, and only in the second case is it cut, after its last caseless letter: the upper-case
//   letter starts a piece exactly when only upper-case letters follow up to the end of the run.
//   A mark at either end of the look leaves the case to the sparse path, and so does leaving the tile.
TT_HD int tt_resolve_upper_after_caseless(const u16 (*sm)[TT_SLOTS], int s, int i) {
    u32 keep = (1u << i) - 1;
    for (int t = s;; t--, keep = 0xFFFFu) {
        if (t < 0) return -1;
        const u32 c = sm[F_CLESS][t], d = sm[F_DOC][t];
        const u32 stop = ((~c & 0xFFFFu) | d) & keep;
        if (!stop) continue;
        const int k = tt_hibit(stop);
        if ((c >> k) & 1) break;                                  // a caseless letter that starts a document
        if ((sm[F_MARK][t] >> k) & 1) return -1;
        if ((sm[F_LOW][t] >> k) & 1) {
            const u32 ap = ((u32)sm[F_AP][t] << 16) | (t > 0 ? (u32)sm[F_AP][t - 1] : 0xFFFFu);
            if ((ap >> (14 + k)) & 3) return -1;                  // apostrophe one or two bytes before it
            return 1;
        }
        break;
    }
    keep = ~((2u << i) - 1) & 0xFFFFu;
    for (int t = s;; t++, keep = 0xFFFFu) {
        if (t >= TT_SLOTS) return -1;
        const u32 u = sm[F_UPP][t], d = sm[F_DOC][t];
        const u32 stop = ((~u & 0xFFFFu) | d) & keep;
        if (!stop) continue;
        const int k = tt_lobit(stop);
        if ((d >> k) & 1) return 1;
        if ((sm[F_MARK][t] >> k) & 1) return -1;
        return (((u32)sm[F_LOW][t] | sm[F_CLESS][t]) >> k) & 1 ? 0 : 1;
    }
}

// An apostrophe between letters (tile position pos = slot * 16 + bit) that has another apostrophe two or three bytes
// before it: is it the start of a contraction suffix of the word in front of it?  1 = yes, 0 = no, -1 = left to the
// sparse path.  A contraction suffix ends its match, so the letter in front of this apostrophe belongs to a word
// body -- and the apostrophe can open a suffix -- unless that letter is itself the last letter of a suffix opened by
// the apostrophe before.  Whether that one opened a suffix hangs on the one before it in the same way: the chain of
// apostrophes is followed to its head (an apostrophe with none two or three bytes before it, or one that is not
// between letters) and decided from there.  base0 / g0: the text and the position of byte 0 of slot 0.
TT_HD int tt_resolve_chained_apostrophe(const u16 (*sm)[TT_SLOTS], int pos, const u8* base, long long g0, long long hi) {
    const int K = 8;
    int chain[K];
    int n = 0;
#define MB(f, q) ((sm[f][(q) >> 4] >> ((q) & 15)) & 1u)
#define LETTER(q) (MB(F_LOW, q) | MB(F_UPP, q) | MB(F_CLESS, q))
#define CAND(q) (MB(F_AP, q) && LETTER((q) - 1) && !MB(F_DOC, q) && LETTER((q) + 1) && !MB(F_DOC, (q) + 1))
    int cur = pos;
    for (;;) {
        if (n == K) return -1;
        if (cur < 4 || cur + 2 >= TT_SLOTS * 16) return -1;       // the look leaves the tile's window
        chain[n++] = cur;
        if (!CAND(cur)) break;                                      // opens no suffix whatever precedes it: a head
        int prev = -1;
        if (MB(F_AP, cur - 2) && !MB(F_DOC, cur - 1) && !MB(F_DOC, cur)) prev = cur - 2;
        else if (MB(F_AP, cur - 3) && !MB(F_DOC, cur - 2) && !MB(F_DOC, cur - 1) && !MB(F_DOC, cur)) prev = cur - 3;
        if (prev < 0) break;                                        // nothing before it can have taken its letter: a head
        cur = prev;
    }
    bool consumed = false;                                          // the letter before the apostrophe ends a suffix
    for (int k = n - 1;; k--) {
        const int q = chain[k];
        int cl = 0;
        if (CAND(q) && !consumed) {
            const long long g = g0 + q;
            const u32 b1 = (g + 1 < hi) ? base[g + 1] : 0, b2 = (g + 2 < hi && !MB(F_DOC, q + 2)) ? base[g + 2] : 0;
            cl = tt_contraction_len(b1, b2);
        }
        if (k == 0) return cl ? 1 : 0;
        consumed = cl != 0 && q + cl == chain[k - 1];
    }
#undef CAND
#undef LETTER
#undef MB
}

// Valid for 1 <= s <= TT_SLOTS - 2 (needs the neighbouring slots).  Unresolved constructs of the second and third
// kind that the tile's masks decide leave `hard`; upper-case letters that start a piece join `sure`.
TT_HD void tt_sure_hard(const u16 (*sm)[TT_SLOTS], int s, u32& sure, u32& hard, const u8* base, long long g0, long long hi) {
    u32 upcl, apch;
    tt_sure_hard_cm(tt_load_slot(sm, s - 1), tt_load_slot(sm, s), tt_load_slot(sm, s + 1), sure, hard, upcl, apch);
    while (upcl) {
        const int i = tt_lobit(upcl);
        upcl &= upcl - 1;
        const int r = tt_resolve_upper_after_caseless(sm, s, i);
        if (r >= 0) { hard &= ~(1u << i); sure |= (u32)r << i; }
    }
    while (apch) {
        const int i = tt_lobit(apch);
        apch &= apch - 1;
        if (tt_resolve_chained_apostrophe(sm, s * 16 + i, base, g0, hi) >= 0) hard &= ~(1u << i);
    }
}

// Walks down from slot s over the precomputed F_SURE / F_HARD masks (valid for slots >= 1): is the
// nearest sure-start / unresolved-construct event an unresolved one?
TT_HD u32 tt_walk_back_dirty(const u16 (*sm)[TT_SLOTS], int s, bool& open) {
    open = false;
    for (; s >= 1; s--) {
        const u32 c = sm[F_SURE][s], h = sm[F_HARD][s];
        if (c | h) { int b = tt_hibit(c | h); return (h >> b) & 1; }
    }
    open = true;
    return 0;
}
// Do the slots 1..s hold neither letters nor marks?  Then no unresolved construct that lies before them can reach beyond
// them: whitespace, punctuation and digits are split by rules that look at most a few bytes back (plus the run
// aggregates that have carries of their own), so what an earlier word turned out to be is forgotten after the first
// such character.  (Asked only by chunks that found no event in the whole look-back window: long runs of blanks or
// of one punctuation character, where the alternative is a walk back to the run's start from every tile in it.)
TT_HD bool tt_window_plain(const u16 (*sm)[TT_SLOTS], int s) {
    u32 wordy = 0;
    for (; s >= 1; s--) wordy |= (u32)sm[F_LOW][s] | sm[F_UPP][s] | sm[F_CLESS][s] | sm[F_MARK][s];
    return wordy == 0;
}
// Walks down from slot s: position (slot * 16 + bit) of the nearest sure start, or -1 when open.
TT_HD int tt_walk_back_sure(const u16 (*sm)[TT_SLOTS], int s) {
    for (; s >= 1; s--) {
        const u32 c = sm[F_SURE][s];
        if (c) return s * 16 + tt_hibit(c);
    }
    return -1;
}
// Is the '/' run that ends at bit `top` of slot s part of a punctuation tail (absorbed)?
// need_a: the answer hangs on a CR/LF run that leaves the window (then the tile carry decides).
TT_HD u32 tt_walk_back_slash(const u16 (*sm)[TT_SLOTS], int s, int top, bool& open_s, bool& open_a) {
    open_s = open_a = false;
    u32 keep = 0xFFFFu >> (15 - top);
    for (; s >= 0; s--, keep = 0xFFFFu) {
        u32 sl = sm[F_SL][s], d = sm[F_DOC][s];
        u32 cut = ((~sl & 0xFFFFu) | (d >> 1)) & keep;
        if (cut) {
            int b = tt_hibit(cut);
            if (((d >> 1) >> b) & 1) return 0;                  // the run starts a document
            if (!((sm[F_NL][s] >> b) & 1)) return 0;            // not preceded by CR/LF
            return tt_walk_back_nl(sm, s, 0, open_a, b);
        }
        if (d & 1) return 0;
    }
    open_s = true;
    return 0;
}

TT_HD u64 tt_win4(const u16 (*sm)[TT_SLOTS], int f, int slot) {   // slots slot-2 .. slot+1; own chunk at bits 32..47
    return (u64)sm[f][slot - 2] | ((u64)sm[f][slot - 1] << 16) | ((u64)sm[f][slot] << 32) | ((u64)sm[f][slot + 1] << 48);
}

// Returns the 16 start bits of the chunk in `slot` (slot >= 2).
TT_HD u32 tt_eval_chunk_p1(const u16 (*sm)[TT_SLOTS], int slot, const SeqCtx& C, long long g0,
                           const TileCarry& tc, bool have_tc, u32& need) {
    const u64 OWN = 0xFFFFull << 32;
    const u64 lead = tt_win4(sm, F_LEAD, slot);
    const u64 low = tt_win4(sm, F_LOW, slot), upp = tt_win4(sm, F_UPP, slot), cless = tt_win4(sm, F_CLESS, slot);
    const u64 Lr = low | upp | cless, Mk = tt_win4(sm, F_MARK, slot);
    const u64 N = tt_win4(sm, F_NUM, slot), W = tt_win4(sm, F_SPC, slot), O = tt_win4(sm, F_OTH, slot);
    const u64 NL = tt_win4(sm, F_NL, slot), SP = tt_win4(sm, F_SP, slot), AP = tt_win4(sm, F_AP, slot), SL = tt_win4(sm, F_SL, slot);
    const u64 D = tt_win4(sm, F_DOC, slot);
    const u64 V = Lr | Mk | N | W | O;
    const u64 cont = V & ~lead;
    const u64 nD = ~D;
    u64 S = 0;
#define PREV(x) (((x) << 1) & nD)
    // ---- CR/LF absorbed by a preceding punctuation character (any non-mark "other", slashes included)
    u64 A;
    {
        u32 carry = 0;
        if ((NL & 1) && !(D & 1)) {                      // the run may enter the window from below
            bool open = slot < 3;
            if (!open) {
                u32 prevnl = (sm[F_NL][slot - 3] >> 15) & 1, prevo = (sm[F_OTH][slot - 3] >> 15) & 1;
                if (prevnl) carry = tt_walk_back_nl(sm, slot - 3, 0, open);
                else carry = prevo;
            }
            if (open) { if (have_tc) carry = tc.nl_absorbed_before; else need |= NEED_A; }
        }
        const u64 nlq = NL & nD;
        const u64 sel = (NL & ~PREV(NL) & PREV(O)) | ((nlq & 1) ? (u64)carry : 0);
        A = nlq & ~(nlq + sel);
    }
    // ---- slashes absorbed by the tail [\r\n/]* : '/' runs that begin right after an absorbed CR/LF
    u64 AS;
    {
        u32 carry = 0;
        if ((SL & 1) && !(D & 1)) {
            bool open_s = slot < 3, open_a = false;
            if (!open_s) {
                u32 prevsl = (sm[F_SL][slot - 3] >> 15) & 1, prevnl = (sm[F_NL][slot - 3] >> 15) & 1;
                if (prevsl) carry = tt_walk_back_slash(sm, slot - 3, 15, open_s, open_a);
                else if (prevnl) carry = tt_walk_back_nl(sm, slot - 3, 0, open_a);
            }
            if (open_s) { if (have_tc) carry = tc.slash_absorbed_before; else need |= NEED_S; }
            if (open_a) { if (have_tc) carry = tc.nl_absorbed_before; else need |= NEED_A; }
        }
        const u64 slq = SL & nD;
        const u64 sel = (SL & ~PREV(SL) & PREV(A)) | ((slq & 1) ? (u64)carry : 0);
        AS = slq & ~(slq + sel);
    }
    // ---- punctuation: a run start that no blank precedes; an absorbed slash is no start and ends the run before it
    const u64 Oe = O & ~AS;
    const u64 G = Oe & lead & ~PREV(Oe) & ~PREV(SP);
    S |= G;
    // ---- words: run start unless non-CR/LF whitespace or a single match-start punctuation char is the prefix
    const u64 c1 = cont << 1, c2 = cont << 2, c3 = cont << 3;
    const u64 pfx = ((G << 1) | ((G << 2) & c1) | ((G << 3) & c2 & c1) | ((G << 4) & c3 & c2 & c1)) & nD;
    S |= Lr & lead & ~PREV(Lr) & ~((PREV(W) & ~PREV(NL)) | pfx);
    S |= upp & lead & PREV(low);                          // case boundary: upper after lower
    // ---- contraction suffix: an apostrophe between letters with a valid suffix ('s 't 'm 'd 're 've 'll, ASCII,
    // any case) belongs to the word before it; the suffix letters start nothing and the next letter starts a piece.
    // (An apostrophe with another one 2-3 bytes before it is decided along the chain of such apostrophes.)
    {
        u64 ca = AP & PREV(Lr) & ((Lr >> 1) & ~(D >> 1)) & (0x7FFFFull << 29);   // own bytes -3 .. +15
        const u64 chained = (AP << 2) | (AP << 3);
        while (ca) {
            const int q = (u32)ca ? tt_lobit((u32)ca) : 32 + tt_lobit((u32)(ca >> 32));
            ca &= ca - 1;
            const long long g = g0 + (q - 32);
            const u32 b1 = (g + 1 < C.hi) ? C.base[g + 1] : 0, b2 = (g + 2 < C.hi) ? C.base[g + 2] : 0;
            int cl = tt_contraction_len(b1, (D >> (q + 2)) & 1 ? 0u : b2);
            // an apostrophe shortly before this one may have taken the letter in front of it: decided along the chain,
            // or (result -1) left to the sparse path, which then overrides these bits
            if (cl && ((chained >> q) & 1) && tt_resolve_chained_apostrophe(sm, (slot - 2) * 16 + q, C.base, g0 - (long long)slot * 16, C.hi) != 1) cl = 0;
            if (cl) {
                const u64 span = ((1ull << cl) - 1) << q;                 // apostrophe and suffix letters
                S &= ~span;
                if (((D >> (q + 1)) & ((1ull << cl) - 1)) == 0) S |= (1ull << (q + cl)) & Lr & lead;
            }
        }
    }
    // ---- number runs: every third lead counted from the run start
    {
        const u32 n_own = (u32)(N >> 32) & 0xFFFFu, ld_own = (u32)(lead >> 32) & 0xFFFFu;
        const u32 nstart = (u32)((N & ~PREV(N)) >> 32) & 0xFFFFu;
        u32 m = n_own & ld_own;
        if (m) {
            u32 cnt = 0;
            if ((n_own & 1) && !(nstart & 1)) {
                bool open;
                cnt = tt_walk_back_num(sm, slot - 1, open);
                if (open) { if (have_tc) cnt += tc.n_before; else need |= NEED_N; }
                cnt %= 3;
            }
            while (m) {
                int i = tt_lobit(m); m &= m - 1;
                if ((nstart >> i) & 1) cnt = 0;
                if (cnt == 0) S |= 1ull << (32 + i);
                cnt = cnt == 2 ? 0 : cnt + 1;
            }
        }
    }
    // ---- whitespace runs (same rules as pattern 0; "punctuation" excludes marks here)
    if (W & OWN) {
        S |= W & lead & ~PREV(W) & ~(PREV(O) & NL);
        S |= W & lead & ~NL & PREV(A);
        const u64 next_exists = (V >> 1) & ~(D >> 1);
        const u64 wend = W & ~((W >> 1) & ~(D >> 1)) & next_exists;
        const u64 k1 = cont >> 1, k2 = cont >> 2, k3 = cont >> 3;
        S |= lead & W & ~NL & (wend | ((wend >> 1) & k1) | ((wend >> 2) & k1 & k2) | ((wend >> 3) & k1 & k2 & k3));
        u32 cand = (u32)((W & lead & ~NL & PREV(NL)) >> 32) & 0xFFFFu;
        while (cand) {
            int i = tt_lobit(cand); cand &= cand - 1;
            bool open;
            u32 later = tt_walk_fwd_nl(sm, slot, i, open);
            if (open) {
                const int raw = tt_raw_fwd_nl(C.base, g0 + (long long)(TT_SLOTS - slot) * TT_CHUNK, C.hi, C.docmask);
                if (raw >= 0) later = (u32)raw;
                else if (have_tc) later = tc.nl_later_after;
                else { need |= NEED_F; later = 1; }
            }
            if (!later) S |= 1ull << (32 + i);
        }
    }
    // ---- unresolved constructs: propagate from each one up to the next sure start
    // sure starts / unresolved constructs of slot-1 and of the own slot (filled in after classification)
    const u64 sure = ((u64)sm[F_SURE][slot - 1] << 16) | ((u64)sm[F_SURE][slot] << 32);
    const u64 hard = ((u64)sm[F_HARD][slot - 1] << 16) | ((u64)sm[F_HARD][slot] << 32);
    // Window bits 0..15 (slot-2) lack look-back at bit 0, so events there are taken from the walk,
    // which starts at slot-2 and has full neighbour information; propagation runs over bits 16..63.
    u64 dirty;
    {
        u32 carry = 0;
        bool open;
        carry = tt_walk_back_dirty(sm, slot - 2, open);
        // (nothing lies before the text: its first tile needs no look beyond the window)
        const bool at_text_start = C.lo >= g0 - (long long)(slot - 1) * TT_CHUNK;
        if (open && !at_text_start && !tt_window_plain(sm, slot - 2)) { if (have_tc) carry = tc.dirty_before; else need |= NEED_H; }
        const u64 sure2 = sure & ~0xFFFFull;
        u64 F = (hard & ~0xFFFFull) | (((u64)carry << 16) & ~sure2);
        u64 R = ~sure2;
        F |= (F << 1) & R;  R &= R << 1;
        F |= (F << 2) & R;  R &= R << 2;
        F |= (F << 4) & R;  R &= R << 4;
        F |= (F << 8) & R;  R &= R << 8;
        F |= (F << 16) & R; R &= R << 16;
        F |= (F << 32) & R;
        dirty = F;
    }
    u32 pending = (u32)((dirty & OWN & V) >> 32) & 0xFFFFu;
    u32 res = (u32)(((S | sure) & lead & OWN) >> 32) & 0xFFFFu;     // sure starts include the decided case boundaries
    while (pending) {
        // re-derive from the last sure start at or below the first unresolved byte, up to the end of
        // the chunk or of the document, whichever comes first
        const int first = tt_lobit(pending) + 32;
        const u64 below = sure & ((2ull << first) - 1) & ~0xFFFFull;
        long long from = -1;
        if (below) {
            int hb = (below >> 32) ? 32 + tt_hibit((u32)(below >> 32)) : tt_hibit((u32)below);
            from = g0 + (hb - 32);
        } else {
            int pos = tt_walk_back_sure(sm, slot - 2);
            if (pos >= 0) from = g0 + ((long long)pos - (long long)slot * 16);
            else if (C.lo >= g0 - (long long)(slot - 1) * TT_CHUNK) from = C.lo;      // the text start is a sure start
            else if (have_tc) from = tc.sure_before;
            else need |= NEED_C;
        }
        if (from < 0) break;
        long long doc_end;
        const u32 seq = tt_seq_starts_p1(C, from, g0, doc_end);
        const int fb = from > g0 ? (int)(from - g0) : 0;
        const int eb = doc_end - g0 >= 16 ? 16 : (int)(doc_end - g0);
        const u32 take = (0xFFFFu << fb) & ~(eb >= 16 ? 0u : (0xFFFFu << eb)) & 0xFFFFu;
        res = (res & ~take) | (seq & take);
        pending &= ~take;
        pending &= ~((1u << (first - 32)) | ((1u << (first - 32)) - 1));     // always make progress
    }
    return res;
#undef PREV
}

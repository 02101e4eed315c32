// Steps K2 and K3: run-local piece-start rules and stream compaction.
//
// Paper Sec. 4.1: whether a character begins a piece depends only on its offset within its
// maximal same-class run, a few characters of look-back across the run boundary, and per-run
// aggregates of whitespace runs (run start, first non-CR/LF position, last CR/LF position); the
// test is an independent per-character predicate.  Here one thread evaluates the predicate for the
// 16 bytes of its chunk as bit-parallel operations on class masks (bit i <-> byte i) over a 48-byte
// window (previous, own, next chunk).  Aggregates that reach further (offset mod 3 inside a number
// run, CR/LF runs glued to preceding punctuation, "is there a CR/LF later in this whitespace run")
// are resolved by walking chunk summaries in shared memory and, beyond the tile, by a bounded
// CTA-cooperative walk over the text itself -- no CTA ever waits for another CTA.
#pragma once
#include "tt_classify.cuh"

enum { F_LEAD = 0, F_OTH, F_MARK, F_SPC, F_NUM, F_LOW, F_UPP, F_CLESS, F_NL, F_SP, F_AP, F_SL, F_DOC,
       F_SURE, F_HARD,     // pattern 1: sure piece starts / unresolved constructs, filled after classification
       F_COUNT };
constexpr int TT_LOW_HALO = 14;                         // chunks kept below the tile (look-back context, 224 bytes)
constexpr int TT_SLOTS = TT_TILE_CHUNKS + TT_LOW_HALO + 1;   // low halo, tile, one high halo chunk

enum { NEED_N = 1, NEED_A = 2, NEED_F = 4, NEED_S = 8, NEED_H = 16, NEED_C = 32 };

struct PretokParams {
    const u8* base;          // 16-byte aligned address at or below the text
    const u8* src;           // null, or the same frame in pinned host memory that the device can read: the kernel then takes the
    u8* copy;                // text from there and leaves a copy of every chunk at `copy` (= base) for all that reads the text later
    long long lo, hi;        // the text occupies [lo, hi) in the aligned frame
    long long nchunks;       // ceil(hi / 16)
    int ntiles;
    int pattern;
    const u32* docmask;      // bit per byte (aligned frame) marking document starts, or null (one document)
    const u32* litstart;     // literal pass: first bytes of extracted literals (each becomes exactly one piece), or null
    const u32* litin;        //               their other bytes (start nothing)
    u16* startmask;          // out (flags-only kernel): one u16 per chunk
    u32* tile_cnt;           // out: pieces per tile; flags-only kernel with want_prefix: replaced by the exclusive prefix (ntiles + 1)
    u32* tile_first;         // out: offset inside the tile of its first piece start, or ~0 if it has none
    int want_prefix;         // turn tile_cnt into its exclusive prefix and count the pieces (tt_pretokenize only)
    TTHeader* hdr;
    unsigned long long epoch; // of this call (see TTHeader)
    const u8* cls_tables;    // stage1 | stage2 | ascii, contiguous in global memory
    int cls_bytes;
};

struct TileCarry {           // aggregates of runs that enter or leave the shared-memory window
    u32 n_before;            // number leads (mod 3) of the number run ending right before the low halo chunk
    u32 nl_absorbed_before;  // the CR/LF run ending right before the low halo chunk is glued to punctuation
    u32 nl_later_after;      // the whitespace run leaving the high halo chunk still contains a CR/LF
    u32 slash_absorbed_before;   // pattern 1: the '/' run ending right before the low halo is part of a punctuation tail
    u32 dirty_before;        // pattern 1: an unresolved construct lies between the last sure piece start and the low halo
    long long sure_before;   // pattern 1: position (aligned frame) of the last sure piece start before the low halo
};

TT_HD u64 tt_win(const u16 (*sm)[TT_SLOTS], int f, int slot) {
    return (u64)sm[f][slot - 1] | ((u64)sm[f][slot] << 16) | ((u64)sm[f][slot + 1] << 32);
}

TT_HD int tt_hibit(u32 x) {   // position of the highest set bit, x != 0
#if defined(__CUDA_ARCH__)
    return 31 - __clz(x);
#else
    return 31 - __builtin_clz(x);
#endif
}
TT_HD int tt_lobit(u32 x) {   // position of the lowest set bit, x != 0
#if defined(__CUDA_ARCH__)
    return __ffs(x) - 1;
#else
    return __builtin_ctz(x);
#endif
}
TT_HD int tt_popc(u32 x) {
#if defined(__CUDA_ARCH__)
    return __popc(x);
#else
    return __builtin_popcount(x);
#endif
}

// ---- run summaries of the window's slots -----------------------------------------------------------------------
// Kept behind the class masks in shared memory: per summary five words, a bit per slot that says "all sixteen bytes
// are ASCII digits" (summary 0) or "all are blanks other than CR/LF" (summary 1), with no document start among them.
// Words 0..3: the tile's own slots (bit = thread), word 4: the low halo slots (bits 0..13), the high one (bit 14) and,
// in bit 31, whether the summary is filled at all (the kernel for bulk text leaves it empty).
// A walk through a run that fills whole tiles -- a number of twenty thousand digits, 64 KB of blanks -- steps over
// such slots at once instead of visiting them one by one from every chunk of the tile.
constexpr int TT_RUNMASK_WORDS = TT_TILE_CHUNKS / 32 + 1;
constexpr int TT_RUNMASK_OFFSET = (int)((sizeof(u16) * F_COUNT * TT_SLOTS + 15) / 16 * 16);      // bytes from the start of the masks
constexpr int TT_PRETOK_SMEM_BYTES = TT_RUNMASK_OFFSET + 2 * TT_RUNMASK_WORDS * (int)sizeof(u32);
TT_HD const u32* tt_runmask(const u16 (*sm)[TT_SLOTS], int which) {
    return reinterpret_cast<const u32*>(reinterpret_cast<const u8*>(sm) + TT_RUNMASK_OFFSET) + which * TT_RUNMASK_WORDS;
}
// highest slot t <= s whose bit is clear (-1: none)
TT_HD int tt_run_skip_back(const u32* rm, int s) {
    constexpr int HW = TT_TILE_CHUNKS / 32;
    if (s >= TT_LOW_HALO + TT_TILE_CHUNKS) { if (!((rm[HW] >> TT_LOW_HALO) & 1)) return s; s = TT_LOW_HALO + TT_TILE_CHUNKS - 1; }
    if (s >= TT_LOW_HALO) {
        const int idx = s - TT_LOW_HALO;
        for (int w = idx >> 5; w >= 0; w--) {
            u32 clear = ~rm[w];
            if (w == (idx >> 5)) clear &= 0xFFFFFFFFu >> (31 - (idx & 31));
            if (clear) return TT_LOW_HALO + w * 32 + tt_hibit(clear);
        }
        s = TT_LOW_HALO - 1;
    }
    const u32 clear = ~rm[HW] & (0xFFFFFFFFu >> (31 - s)) & ((1u << TT_LOW_HALO) - 1);
    return clear ? tt_hibit(clear) : -1;
}
// lowest slot t >= s whose bit is clear (TT_SLOTS: none)
TT_HD int tt_run_skip_fwd(const u32* rm, int s) {
    constexpr int HW = TT_TILE_CHUNKS / 32;
    if (s >= TT_SLOTS) return TT_SLOTS;
    if (s < TT_LOW_HALO) {
        const u32 clear = ~rm[HW] & ((1u << TT_LOW_HALO) - 1) & (0xFFFFFFFFu << s);
        if (clear) return tt_lobit(clear);
        s = TT_LOW_HALO;
    }
    if (s < TT_LOW_HALO + TT_TILE_CHUNKS) {
        const int idx = s - TT_LOW_HALO;
        for (int w = idx >> 5; w < HW; w++) {
            u32 clear = ~rm[w];
            if (w == (idx >> 5)) clear &= 0xFFFFFFFFu << (idx & 31);
            if (clear) return TT_LOW_HALO + w * 32 + tt_lobit(clear);
        }
    }
    return ((rm[HW] >> TT_LOW_HALO) & 1) ? TT_SLOTS : TT_SLOTS - 1;
}

// Number leads in the number run that ends at the last byte of slot `s` (walking down).
// Returns the count; sets `open` when the run continues below slot 0.
TT_HD u32 tt_walk_back_num(const u16 (*sm)[TT_SLOTS], int s, bool& open) {
    u32 cnt = 0;
    open = false;
    const u32* rm = tt_runmask(sm, 0);
    const bool summaries = (rm[TT_TILE_CHUNKS / 32] >> 31) != 0;
    for (; s >= 0; s--) {
        if (summaries) {
            int t = tt_run_skip_back(rm, s);                // slots of sixteen ASCII digits: sixteen leads each
            if (t > s) t = s;                               // (never upwards: the loop ends whatever the summary holds)
            cnt += 16u * (u32)(s - t);
            s = t;
            if (s < 0) break;
        }
        u32 n = sm[F_NUM][s], d = sm[F_DOC][s], ld = sm[F_LEAD][s];
        u32 cut = (~n & 0xFFFFu) | (d >> 1);        // byte j ends the walk if it is not a number byte or j+1 starts a document
        if (cut) { int b = tt_hibit(cut); cnt += tt_popc(ld & n & (0xFFFFu << (b + 1)) & 0xFFFFu); return cnt; }
        cnt += tt_popc(ld & n);
        if (d & 1) return cnt;                      // run starts at a document start
    }
    open = true;
    return cnt;
}

// Is the CR/LF run that ends at the last byte of slot `s` glued to a preceding punctuation char?
// (0 / 1; `open` when the run continues below slot 0.)
TT_HD u32 tt_walk_back_nl(const u16 (*sm)[TT_SLOTS], int s, u32 othmask_fields, bool& open, int top = 15) {
    open = false;
    u32 keep = 0xFFFFu >> (15 - top);               // the walk starts at bit `top` of slot s
    for (; s >= 0; s--, keep = 0xFFFFu) {
        u32 nl = sm[F_NL][s], d = sm[F_DOC][s];
        u32 cut = ((~nl & 0xFFFFu) | (d >> 1)) & keep;
        if (cut) {
            int b = tt_hibit(cut);
            if ((d >> 1) >> b & 1) return 0;        // the run starts at a document start
            u32 o = sm[F_OTH][s] | (othmask_fields ? sm[F_MARK][s] : 0);
            return (o >> b) & 1;
        }
        if (d & 1) return 0;
    }
    open = true;
    return 0;
}

// Does the whitespace run that contains byte `bit` of slot `s` contain a CR/LF above that byte?
TT_HD u32 tt_walk_fwd_nl(const u16 (*sm)[TT_SLOTS], int s, int bit, bool& open) {
    open = false;
    u32 low = (0xFFFFu << (bit + 1)) & 0xFFFFu;
    const u32* rm = tt_runmask(sm, 1);
    const bool summaries = (rm[TT_TILE_CHUNKS / 32] >> 31) != 0;
    for (; s < TT_SLOTS; s++) {
        u32 w = sm[F_SPC][s], nl = sm[F_NL][s], d = sm[F_DOC][s];
        u32 ev = ((~w) | d | nl) & low;
        if (ev) { int j = tt_lobit(ev); return ((nl & w & ~d) >> j) & 1; }
        low = 0xFFFFu;
        if (summaries) {
            const int t = tt_run_skip_fwd(rm, s + 1);       // slots of sixteen plain blanks hold no event
            if (t > s + 1) s = t - 1;                       // (never backwards: the loop ends whatever the summary holds)
        }
    }
    open = true;
    return 0;
}

// The same question asked of the raw text from byte g on (the run has left the shared-memory window):
// 1 / 0 = answered from ASCII bytes alone, -1 = undecided (a non-ASCII byte, which may be whitespace, or more
// than `limit` bytes of blanks).  A document start cuts the run.  One thread, plain loads.
TT_HD int tt_raw_fwd_nl(const u8* base, long long g, long long hi, const u32* docmask, int limit = 256) {
    int k = 0;
    // sixteen bytes at a time while they are all blanks other than CR/LF and no document starts among them (g is a
    // multiple of 16 for every caller; `base` is 16-byte aligned)
    if ((g & 15) == 0) {
        for (; k + 16 <= limit && g + 16 <= hi; k += 16, g += 16) {
            const uint4 v = *reinterpret_cast<const uint4*>(base + g);
            const u32 w[4] = {v.x, v.y, v.z, v.w};
            bool plain = ((v.x | v.y | v.z | v.w) & 0x80808080u) == 0;
            if (docmask) plain = plain && reinterpret_cast<const u16*>(docmask)[g >> 4] == 0;
#pragma unroll
            for (int j = 0; j < 4; j++)
                plain = plain && (tt_swar_range(w[j], 0x09, 0x09) | tt_swar_range(w[j], 0x0B, 0x0C) | tt_swar_range(w[j], ' ', ' ')) == 0x80808080u;
            if (!plain) break;
        }
    }
    for (; k < limit; k++, g++) {
        if (g >= hi) return 0;
        if (docmask && ((docmask[g >> 5] >> (g & 31)) & 1)) return 0;        // the run is cut by a document start
        const u32 b = base[g];
        if (b == '\n' || b == '\r') return 1;
        if (b >= 0x80) return -1;
        if (!(b == ' ' || (b >= 0x09 && b <= 0x0C))) return 0;
    }
    return -1;
}

// Contraction suffix length at the apostrophe whose two following bytes are b1, b2 (0 = none).
TT_HD int tt_contraction_len(u32 b1, u32 b2) {
    const u32 a = b1 | 0x20, b = b2 | 0x20;       // ASCII case fold; no other byte maps onto these letters
    if (a == 's' || a == 't' || a == 'm' || a == 'd') return 2;
    if ((a == 'r' && b == 'e') || (a == 'v' && b == 'e') || (a == 'l' && b == 'l')) return 3;
    return 0;
}

// First two stages of the three-splitter composition (paper Sec. 4.1: three splitters applied in sequence
// fold into the same per-character predicate, provided each splitter re-splits every piece of the stage
// before it and unmatched spans survive as pieces): number groups of up to three digits and runs of
// caseless letters are isolated.  Returns the 16 cut bits of the chunk in `slot`: a bit where a span of
// these two stages begins.  The third stage (pattern 0) then runs with the cuts as document boundaries,
// i.e. on every span as a text of its own.
constexpr int TT_PATTERN_CUTS = 100;              // internal pattern id of this pass
TT_HD u32 tt_eval_chunk_cuts(const u16 (*sm)[TT_SLOTS], int slot, const TileCarry& tc, bool have_tc, u32& need) {
    const u64 OWN = 0xFFFFull << 16;
    const u64 lead = tt_win(sm, F_LEAD, slot), N = tt_win(sm, F_NUM, slot), C = tt_win(sm, F_CLESS, slot), D = tt_win(sm, F_DOC, slot);
    const u64 nD = ~D;
#define PREV(x) (((x) << 1) & nD)
    u64 S = D;
    S |= lead & ~N & PREV(N);                        // first character after a number run
    S |= C & lead & ~PREV(C);                        // a run of caseless letters begins
    S |= lead & ~C & PREV(C);                        // first character after such a run
    const u32 n_own = (u32)(N >> 16) & 0xFFFFu, ld_own = (u32)(lead >> 16) & 0xFFFFu;
    const u32 nstart = (u32)((N & ~PREV(N)) >> 16) & 0xFFFFu;
    u32 m = n_own & ld_own;
    if (m) {                                         // every third number lead counted from the run start
        u32 cnt = 0;
        if ((n_own & 1) && !(nstart & 1)) {
            bool open;
            cnt = tt_walk_back_num(sm, slot - 1, open);
            if (open) { if (have_tc) cnt += tc.n_before; else need |= NEED_N; }
            cnt %= 3;
        }
        while (m) {
            const int i = tt_lobit(m); m &= m - 1;
            if ((nstart >> i) & 1) cnt = 0;
            if (cnt == 0) S |= 1ull << (16 + i);
            cnt = cnt == 2 ? 0 : cnt + 1;
        }
    }
#undef PREV
    return (u32)((S & lead & OWN) >> 16);
}

// A 32-bit window over the masks of field f: bits 0..7 = the last eight bytes of the chunk before, bits 8..23 = the
// chunk in `slot`, bits 24..31 = the first eight bytes of the chunk after it.  Pattern 0 looks at most four bytes
// back and three ahead, so single-word operations cover it.
TT_HD u32 tt_win32(const u16 (*sm)[TT_SLOTS], int f, int slot) {
    return ((u32)sm[f][slot - 1] >> 8) | ((u32)sm[f][slot] << 8) | ((u32)sm[f][slot + 1] << 24);
}

// Pattern 0 (cl100k-style).  Returns the 16 start bits of the chunk in `slot`; `need` receives the
// NEED_* flags of aggregates that leave the shared-memory window (then `tc` must be filled and the
// function called again).
TT_HD u32 tt_eval_chunk_p0(const u16 (*sm)[TT_SLOTS], int slot, const u8* base, long long g0, long long hi,
                           const TileCarry& tc, bool have_tc, u32& need, bool single_digits = false,
                           const u32* docmask = nullptr) {
    const u32 OWN = 0xFFFFu << 8;
    const u32 lead = tt_win32(sm, F_LEAD, slot);
    const u32 L = tt_win32(sm, F_LOW, slot) | tt_win32(sm, F_UPP, slot) | tt_win32(sm, F_CLESS, slot);
    const u32 N = tt_win32(sm, F_NUM, slot);
    const u32 W = tt_win32(sm, F_SPC, slot);
    const u32 O = tt_win32(sm, F_OTH, slot) | tt_win32(sm, F_MARK, slot);
    const u32 NL = tt_win32(sm, F_NL, slot), SP = tt_win32(sm, F_SP, slot), AP = tt_win32(sm, F_AP, slot);
    const u32 D = tt_win32(sm, F_DOC, slot);
    const u32 V = L | N | W | O;                       // bytes that exist and are valid
    const u32 cont = V & ~lead;
    const u32 nD = ~D;
    u32 S = 0;
#define PREV(x) (((x) << 1) & nD)
    // punctuation runs: start of the run, unless a blank precedes it (the blank starts the piece)
    const u32 G = O & lead & ~PREV(O) & ~PREV(SP);
    S |= G;
    // letter runs: the run start, unless non-CR/LF whitespace or a single match-start punctuation char precedes it
    const u32 c1 = cont << 1, c2 = cont << 2, c3 = cont << 3;
    const u32 pfx = ((G << 1) | ((G << 2) & c1) | ((G << 3) & c2 & c1) | ((G << 4) & c3 & c2 & c1)) & nD;
    S |= L & lead & ~PREV(L) & ~((PREV(W) & ~PREV(NL)) | pfx);
    // contractions: apostrophe that is a match start, then s/t/m/d or re/ve/ll; the letter after the suffix starts a piece
    u32 ga = G & AP & (0x3FFFFu << 4);                 // apostrophes at own bytes -4 .. +13 can put a start into this chunk
    while (ga) {
        const int p = tt_lobit(ga); ga &= ga - 1;
        const long long g = g0 + (p - 8);
        u32 b1 = (g + 1 < hi) ? base[g + 1] : 0, b2 = (g + 2 < hi) ? base[g + 2] : 0;
        if ((D >> (p + 1)) & 1) b1 = 0;
        if ((D >> (p + 2)) & 1) b2 = 0;
        const int cl = tt_contraction_len(b1, b2);
        if (cl) {
            const u32 at = 1u << (p + cl);
            const bool same_doc = ((D >> (p + 1)) & ((1u << cl) - 1)) == 0;
            if (same_doc) S |= at & L & lead;
        }
    }
    // number runs: every third number lead counted from the run start (single-digit variant: every lead)
    if (single_digits) S |= N & lead;
    else {
        const u32 n_own = (N >> 8) & 0xFFFFu, ld_own = (lead >> 8) & 0xFFFFu;
        const u32 nstart = ((N & ~PREV(N)) >> 8) & 0xFFFFu;
        u32 m = n_own & ld_own;
        if (m) {
            u32 cnt = 0;
            if ((n_own & 1) && !(nstart & 1)) {            // the run enters from the previous chunk
                bool open;
                cnt = tt_walk_back_num(sm, slot - 1, open);
                if (open) { if (have_tc) cnt += tc.n_before; else need |= NEED_N; }
                cnt %= 3;
            }
            while (m) {
                const int i = tt_lobit(m); m &= m - 1;
                if ((nstart >> i) & 1) cnt = 0;
                if (cnt == 0) S |= 1u << (8 + i);
                cnt = cnt == 2 ? 0 : cnt + 1;
            }
        }
    }
    // whitespace runs
    if (W & OWN) {
        // (a) run start, unless it is a CR/LF glued to preceding punctuation
        S |= W & lead & ~PREV(W) & ~(PREV(O) & NL);
        // (b) CR/LF absorbed by preceding punctuation: CR/LF runs that begin right after punctuation
        const u32 nl_own = (NL >> 8) & 0xFFFFu, d_own = (D >> 8) & 0xFFFFu;
        u32 prev_absorbed = 0;                             // byte before the chunk is an absorbed CR/LF
        if (((NL >> 7) & 1) && !(d_own & 1)) {
            bool open;
            prev_absorbed = tt_walk_back_nl(sm, slot - 1, 1, open);
            if (open) { if (have_tc) prev_absorbed = tc.nl_absorbed_before; else need |= NEED_A; }
        }
        const u32 nlq = nl_own & ~d_own;
        const u32 sel = (((NL & ~PREV(NL) & PREV(O)) >> 8) & 0xFFFFu) | ((nlq & 1) ? prev_absorbed : 0);
        const u32 absorbed = nlq & ~(nlq + sel);
        const u32 prevA = ((absorbed << 9) | (prev_absorbed << 8)) & nD;
        S |= W & lead & ~NL & prevA;
        // (c) last character of the run when something follows in the same document (and it is not CR/LF)
        const u32 next_exists = (V >> 1) & ~(D >> 1);
        const u32 wend = W & ~((W >> 1) & ~(D >> 1)) & next_exists;
        const u32 k1 = cont >> 1, k2 = cont >> 2, k3 = cont >> 3;
        S |= lead & W & ~NL & (wend | ((wend >> 1) & k1) | ((wend >> 2) & k1 & k2) | ((wend >> 3) & k1 & k2 & k3));
        // (d) first character after the last CR/LF of the run
        u32 cand = ((W & lead & ~NL & PREV(NL)) >> 8) & 0xFFFFu;
        while (cand) {
            const int i = tt_lobit(cand); cand &= cand - 1;
            bool open;
            u32 later = tt_walk_fwd_nl(sm, slot, i, open);
            if (open) {
                const int raw = tt_raw_fwd_nl(base, g0 + (long long)(TT_SLOTS - slot) * TT_CHUNK, hi, docmask);
                if (raw >= 0) later = (u32)raw;
                else if (have_tc) later = tc.nl_later_after;
                else { need |= NEED_F; later = 1; }
            }
            if (!later) S |= 1u << (8 + i);
        }
    }
#undef PREV
    return (S & lead & OWN) >> 8;
}

// Step K1: vector loads of UTF-8 text, strict validation, per-code-point class tagging.
//
// One call classifies one aligned 16-byte chunk and returns, for its 16 bytes, one bit per byte
// in each of the masks below.  Continuation bytes carry the class of their lead byte, so that a
// maximal run of one class is contiguous in byte space (paper Sec. 4.1: character classes and
// maximal same-class runs; Sec. 4.2: on-device UTF-8 decoding and character classification).
#pragma once
#include "tt_common.cuh"

struct ClassTables {          // pointers into shared memory on the device
    const u8* stage1;         // [0x1100]  code point >> 8 -> block
    const u8* stage2;         // [nblocks * 128] two 4-bit class codes per byte
    const u8* ascii;          // [128] class code | (flag << 3); flag: 1 CR/LF, 2 blank, 3 apostrophe, 4 slash
};

struct ChunkMasks {
    u16 lead;                 // byte starts a code point
    u16 oth, mark, spc, num, low, upp, cless;   // class of the code point the byte belongs to
    u16 nl, sp, ap, sl;       // CR/LF, U+0020, apostrophe, slash (ASCII, single byte)
    u16 bad;                  // byte takes part in a UTF-8 violation
};

TT_HD u32 tt_class_of(u32 cp, const ClassTables& T) {
    u32 blk = T.stage1[cp >> 8];
    u32 v = T.stage2[blk * 128 + ((cp & 0xFF) >> 1)];
    return (cp & 1) ? (v >> 4) : (v & 15);
}

// Fills the 128-entry ASCII table (used on the host when the vocab is loaded).
inline void tt_fill_ascii_table(u8* t) {
    for (int b = 0; b < 128; b++) {
        u32 code = CC_OTHER;
        if (b >= '0' && b <= '9') code = CC_NUMBER;
        else if (b >= 'a' && b <= 'z') code = CC_LOWER;
        else if (b >= 'A' && b <= 'Z') code = CC_UPPER;
        else if ((b >= 9 && b <= 13) || b == 32) code = CC_SPACE;
        u32 flag = (b == 10 || b == 13) ? 1 : b == 32 ? 2 : b == 39 ? 3 : b == 47 ? 4 : 0;
        t[b] = (u8)(code | (flag << 3));
    }
}

// ---- sixteen ASCII bytes without a table ------------------------------------------------------------------
// For a word of four bytes below 0x80, tt_swar_ge(y, c) has the top bit of a byte set exactly where that byte is
// >= c (1 <= c <= 0x80): the byte-wise sums stay below 0x100, so nothing carries from byte to byte.  A range is
// ge(lo) & ~ge(hi + 1).
TT_HD u32 tt_swar_ge(u32 y, u32 c) { return y + (0x80u - c) * 0x01010101u; }
TT_HD u32 tt_swar_range(u32 y, u32 lo, u32 hi) { return tt_swar_ge(y, lo) & ~tt_swar_ge(y, hi + 1) & 0x80808080u; }
// The four words are first transposed (word j = byte j of each input word), so that the top bits of the test
// results fall into place with four shifts: bit 4k + j of the result <- top bit of byte k of m_j.
TT_HD u32 tt_gather_top_bits(u32 m0, u32 m1, u32 m2, u32 m3) {
    u32 u = (m0 >> 7) | (m1 >> 6) | (m2 >> 5) | (m3 >> 4);          // bit 8k + j
    u = (u | (u >> 4)) & 0x00FF00FFu;
    return (u | (u >> 8)) & 0xFFFFu;
}
TT_HD u32 tt_perm(u32 x, u32 y, u32 sel) {                              // bytes of {x, y} picked by four selector nibbles
#if defined(__CUDA_ARCH__)
    return __byte_perm(x, y, sel);
#else
    const u64 v = ((u64)y << 32) | x;
    u32 r = 0;
    for (int i = 0; i < 4; i++) r |= (u32)((v >> (8 * ((sel >> (4 * i)) & 7))) & 0xFF) << (8 * i);
    return r;
#endif
}
TT_HD ChunkMasks tt_classify_ascii16(u32 w0, u32 w1, u32 w2, u32 w3) {
    // transpose: y[j] = (byte j of w0, byte j of w1, byte j of w2, byte j of w3)
    const u32 p = tt_perm(w0, w1, 0x5140u), q = tt_perm(w2, w3, 0x5140u);      // bytes 0 and 1 of each pair
    const u32 r = tt_perm(w0, w1, 0x7362u), t = tt_perm(w2, w3, 0x7362u);      // bytes 2 and 3
    const u32 y[4] = {tt_perm(p, q, 0x5410u), tt_perm(p, q, 0x7632u), tt_perm(r, t, 0x5410u), tt_perm(r, t, 0x7632u)};
    u32 let[4], cas[4], num[4], spc[4], nl[4], sp[4], ap[4], sl[4], oth[4];
#pragma unroll
    for (int j = 0; j < 4; j++) {
        const u32 v = y[j];
        let[j] = tt_swar_range(v | 0x20202020u, 'a', 'z');                      // only letters fold into a..z
        cas[j] = v << 2;                                                          // bit 5 of a byte (lower case) in its top bit
        num[j] = tt_swar_range(v, '0', '9');
        sp[j] = tt_swar_range(v, ' ', ' ');
        spc[j] = tt_swar_range(v, 9, 13) | sp[j];
        nl[j] = tt_swar_range(v, '\n', '\n') | tt_swar_range(v, '\r', '\r');
        ap[j] = tt_swar_range(v, '\'', '\'');
        sl[j] = tt_swar_range(v, '/', '/');
        oth[j] = ~(let[j] | num[j] | spc[j]) & 0x80808080u;
    }
    ChunkMasks m;
    m.lead = 0xFFFF; m.mark = 0; m.cless = 0; m.bad = 0;
    m.low = (u16)tt_gather_top_bits(let[0] & cas[0], let[1] & cas[1], let[2] & cas[2], let[3] & cas[3]);
    m.upp = (u16)tt_gather_top_bits(let[0] & ~cas[0], let[1] & ~cas[1], let[2] & ~cas[2], let[3] & ~cas[3]);
    m.num = (u16)tt_gather_top_bits(num[0], num[1], num[2], num[3]);
    m.spc = (u16)tt_gather_top_bits(spc[0], spc[1], spc[2], spc[3]);
    m.oth = (u16)tt_gather_top_bits(oth[0], oth[1], oth[2], oth[3]);
    m.nl = (u16)tt_gather_top_bits(nl[0], nl[1], nl[2], nl[3]);
    m.sp = (u16)tt_gather_top_bits(sp[0], sp[1], sp[2], sp[3]);
    m.ap = (u16)tt_gather_top_bits(ap[0], ap[1], ap[2], ap[3]);
    m.sl = (u16)tt_gather_top_bits(sl[0], sl[1], sl[2], sl[3]);
    return m;
}

// Top bits of the four bytes of a word as a 4-bit number (byte k -> bit k): the bits are first brought to positions
// 0, 8, 16, 24; the multiplication then adds them up at 24..27 (the partial products fall on distinct bits).
TT_HD u32 tt_movemask4(u32 x) { return ((((x >> 7) & 0x01010101u) * 0x01020408u) >> 24) & 0xFu; }

// A chunk that holds non-ASCII bytes.  Its ASCII bytes are classified like those of a plain chunk (the other bytes
// blanked out for the purpose); the loop then visits only the lead bytes of multi-byte characters -- those of the
// chunk and those of the three bytes before it, whose characters may reach into the chunk -- decodes, validates and
// looks up each one.  One copy of this code serves every caller (arguments by value: nothing of the caller has to
// live in memory for the call's sake).
// w0..w5 = the 4 bytes before the chunk, the chunk, the 4 bytes after it (missing neighbours are zero); g0 = global
// index (in the aligned frame) of the chunk's first byte; bytes outside [lo, hi) do not exist; valid = the chunk's
// bytes inside [lo, hi).
TT_HD_COLD ChunkMasks tt_classify_words_general(u32 w0, u32 w1, u32 w2, u32 w3, u32 w4, u32 w5, long long g0, long long lo,
                                                long long hi, u32 valid, const u8* stage1, const u8* stage2) {
    const u32 w[7] = {w0, w1, w2, w3, w4, w5, 0u};
    ClassTables T;
    T.stage1 = stage1; T.stage2 = stage2; T.ascii = nullptr;
    // bit k <- byte k of the chunk has its top bit set / has bit 6 set
    const u32 na = tt_movemask4(w1) | (tt_movemask4(w2) << 4) | (tt_movemask4(w3) << 8) | (tt_movemask4(w4) << 12);
    const u32 b6 = tt_movemask4(w1 << 1) | (tt_movemask4(w2 << 1) << 4) | (tt_movemask4(w3 << 1) << 8) | (tt_movemask4(w4 << 1) << 12);
    const u32 ascm = ~na & valid;
    // words with the non-ASCII bytes blanked: a byte whose top bit is set becomes 0
#define TT_BLANK(x) ((x) & ~((((x) >> 7) & 0x01010101u) * 0xFFu))
    ChunkMasks m = tt_classify_ascii16(TT_BLANK(w1), TT_BLANK(w2), TT_BLANK(w3), TT_BLANK(w4));
#undef TT_BLANK
    m.oth &= (u16)ascm; m.spc &= (u16)ascm; m.num &= (u16)ascm; m.low &= (u16)ascm; m.upp &= (u16)ascm;
    m.nl &= (u16)ascm; m.sp &= (u16)ascm; m.ap &= (u16)ascm; m.sl &= (u16)ascm;
    u32 lead = ascm, bad = 0, cov = 0;
    u64 accA = 0, accB = 0;             // 16-bit lanes: A = class codes 0..3, B = codes 4..6
    const u32 contm = na & ~b6 & valid;                           // continuation bytes of the chunk
    // lead bytes: bit (j + 3) for j = -3 .. 15
    u32 todo = ((na & b6) << 3) | ((tt_movemask4(w0) & tt_movemask4(w0 << 1)) >> 1);
    while (todo) {
#if defined(__CUDA_ARCH__)
        const int j = __ffs((int)todo) - 4;
#else
        const int j = __builtin_ctz(todo) - 3;
#endif
        todo &= todo - 1;
        if (g0 + j < lo || g0 + j >= hi) continue;          // the byte does not exist
        const int at = j + 4;                                     // byte index in w
        const u32 sh = (u32)(at & 3) * 8, x0 = w[at >> 2], x1 = w[(at >> 2) + 1];
        const u32 v = sh ? (x0 >> sh) | (x1 << (32 - sh)) : x0;   // the lead byte and the three bytes behind it
        const u32 b = v & 0xFFu, b1 = (v >> 8) & 0xFFu, b2 = (v >> 16) & 0xFFu, b3 = v >> 24;
        const int n = b >= 0xF0 ? 4 : b >= 0xE0 ? 3 : 2;
        if (j + n - 1 < 0) continue;                     // ends before this chunk
        if (j >= 0) lead |= 1u << j;
        bool ok = (b >= 0xC2) && (b <= 0xF4);
        u32 cp = b & (0x7Fu >> n);
        ok = ok && (g0 + j + n - 1 < hi);
        ok = ok && ((b1 & 0xC0) == 0x80);
        cp = (cp << 6) | (b1 & 0x3F);
        if (n >= 3) { ok = ok && ((b2 & 0xC0) == 0x80); cp = (cp << 6) | (b2 & 0x3F); }
        if (n >= 4) { ok = ok && ((b3 & 0xC0) == 0x80); cp = (cp << 6) | (b3 & 0x3F); }
        if (n == 3) ok = ok && cp >= 0x800 && !(cp >= 0xD800 && cp <= 0xDFFF);
        if (n == 4) ok = ok && cp >= 0x10000 && cp <= 0x10FFFF;
        const u32 span = ((((1u << n) - 1) << (j + 3)) >> 3) & 0xFFFFu;   // bytes of this char inside the chunk
        if (!ok) { bad |= span; continue; }
        const u32 c = tt_class_of(cp, T);
        const u64 lane = (u64)span << ((c & 3) * 16);
        accA |= (c < 4) ? lane : 0ull;
        accB |= (c >= 4) ? lane : 0ull;
        cov |= span;
    }
    bad |= contm & ~cov;                                 // continuation byte without a lead
    m.lead = (u16)(lead & valid);
    m.oth |= (u16)(accA & valid);          m.mark = (u16)((accA >> 16) & valid);
    m.spc |= (u16)((accA >> 32) & valid);  m.num |= (u16)((accA >> 48) & valid);
    m.low |= (u16)(accB & valid);          m.upp |= (u16)((accB >> 16) & valid);
    m.cless = (u16)((accB >> 32) & valid);
    m.bad = (u16)(bad & valid);
    return m;
}

// `w` = the 4 bytes before the chunk, the chunk, the 4 bytes after it; g0, lo, hi as above.
TT_HD ChunkMasks tt_classify_words(const u32 (&w)[6], long long g0, long long lo, long long hi, const ClassTables& T) {
    // bytes of the chunk inside [lo, hi)
    const long long vlo = lo - g0, vhi = hi - g0;
    const u32 klo = vlo <= 0 ? 0u : vlo >= 16 ? 16u : (u32)vlo, khi = vhi <= 0 ? 0u : vhi >= 16 ? 16u : (u32)vhi;
    const u32 valid = khi > klo ? ((1u << khi) - 1u) & ~((1u << klo) - 1u) : 0u;
    const bool all_ascii = ((w[1] | w[2] | w[3] | w[4]) & 0x80808080u) == 0;
    if (!all_ascii) return tt_classify_words_general(w[0], w[1], w[2], w[3], w[4], w[5], g0, lo, hi, valid, T.stage1, T.stage2);
    // sixteen ASCII bytes at once: byte-wise range tests on the four words (see tt_swar_ge), the flag bits gathered
    // into 16-bit masks; no table look-ups
    ChunkMasks a = tt_classify_ascii16(w[1], w[2], w[3], w[4]);
    a.lead = (u16)(0xFFFFu & valid);
    a.oth &= (u16)valid; a.spc &= (u16)valid; a.num &= (u16)valid; a.low &= (u16)valid; a.upp &= (u16)valid;
    a.nl &= (u16)valid; a.sp &= (u16)valid; a.ap &= (u16)valid; a.sl &= (u16)valid;
    return a;
}

// Classifies chunk `chunk`, whose sixteen bytes the caller has loaded (v; zero for a chunk outside [0, nchunks)); the
// two 4-byte neighbours are fetched with aligned accesses where they matter.  `base` is 16-byte aligned.
TT_HD ChunkMasks tt_classify_chunk_loaded(const uint4 v, const u8* base, long long chunk, long long nchunks, long long lo, long long hi,
                                          const ClassTables& T) {
    u32 w[6] = {0, v.x, v.y, v.z, v.w, 0};
    if (chunk >= 0 && chunk < nchunks && ((v.x | v.y | v.z | v.w) & 0x80808080u) != 0) {       // the neighbours matter only to multi-byte characters
        if (chunk > 0) w[0] = *reinterpret_cast<const u32*>(base + chunk * TT_CHUNK - 4);
        if (chunk + 1 < nchunks) w[5] = *reinterpret_cast<const u32*>(base + (chunk + 1) * TT_CHUNK);
    }
    return tt_classify_words(w, chunk * TT_CHUNK, lo, hi, T);
}
// Loads the chunk and classifies it; chunks outside [0, nchunks) are empty.
TT_HD ChunkMasks tt_classify_chunk(const u8* base, long long chunk, long long nchunks, long long lo, long long hi,
                                   const ClassTables& T) {
    uint4 v = make_uint4(0, 0, 0, 0);
    if (chunk >= 0 && chunk < nchunks) v = *reinterpret_cast<const uint4*>(base + chunk * TT_CHUNK);
    return tt_classify_chunk_loaded(v, base, chunk, nchunks, lo, hi, T);
}

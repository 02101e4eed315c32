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

// words w[0] = the 4 bytes before the chunk, w[1..4] = the chunk, w[5] = the 4 bytes after it
#define TT_BYTE(w, j) (((w)[((j) + 4) >> 2] >> (8 * (((j) + 4) & 3))) & 0xFFu)

// g0 = global index (in the aligned frame) of the chunk's first byte; bytes outside [lo, hi) do
// not exist.  `w` as above (missing neighbours are zero).
TT_HD ChunkMasks tt_classify_words(const u32 (&w)[6], long long g0, long long lo, long long hi, const ClassTables& T) {
    u64 accA = 0, accB = 0, accF = 0;   // 16-bit lanes: A = codes 0..3, B = codes 4..6, F = flags 1..4
    u32 lead = 0, bad = 0, cov = 0, contm = 0;
    u32 valid = 0;
#pragma unroll
    for (int k = 0; k < 16; k++) valid |= (u32)(g0 + k >= lo && g0 + k < hi) << k;
    const bool all_ascii = ((w[1] | w[2] | w[3] | w[4]) & 0x80808080u) == 0;
    if (all_ascii) {
#pragma unroll
        for (int k = 0; k < 16; k++) {
            u32 b = TT_BYTE(w, k);
            u32 v = T.ascii[b];
            u32 c = v & 7, f = v >> 3;
            u64 bit = 1ull << ((c & 3) * 16 + k);
            accA |= (c < 4) ? bit : 0ull;
            accB |= (c >= 4) ? bit : 0ull;
            accF |= f ? (1ull << ((f - 1) * 16 + k)) : 0ull;
        }
        lead = 0xFFFF;
    } else {
#pragma unroll
        for (int j = -3; j < 16; j++) {
            u32 b = TT_BYTE(w, j);
            bool exists = (g0 + j >= lo) && (g0 + j < hi);
            if (!exists) continue;
            if (b < 0x80) {
                if (j >= 0) {
                    u32 v = T.ascii[b];
                    u32 c = v & 7, f = v >> 3;
                    u64 bit = 1ull << ((c & 3) * 16 + j);
                    accA |= (c < 4) ? bit : 0ull;
                    accB |= (c >= 4) ? bit : 0ull;
                    accF |= f ? (1ull << ((f - 1) * 16 + j)) : 0ull;
                    lead |= 1u << j;
                }
                continue;
            }
            if ((b & 0xC0) == 0x80) { if (j >= 0) contm |= 1u << j; continue; }
            int n = b >= 0xF0 ? 4 : b >= 0xE0 ? 3 : 2;
            if (j + n - 1 < 0) continue;                     // ends before this chunk
            if (j >= 0) lead |= 1u << j;
            bool ok = (b >= 0xC2) && (b <= 0xF4);
            u32 cp = b & (0x7Fu >> n);
            u32 b1 = (j + 1 < 19) ? TT_BYTE(w, (j + 1 < 19 ? j + 1 : 18)) : 0;
            u32 b2 = (j + 2 < 19) ? TT_BYTE(w, (j + 2 < 19 ? j + 2 : 18)) : 0;
            u32 b3 = (j + 3 < 19) ? TT_BYTE(w, (j + 3 < 19 ? j + 3 : 18)) : 0;
            ok = ok && (g0 + j + n - 1 < hi);
            ok = ok && ((b1 & 0xC0) == 0x80);
            cp = (cp << 6) | (b1 & 0x3F);
            if (n >= 3) { ok = ok && ((b2 & 0xC0) == 0x80); cp = (cp << 6) | (b2 & 0x3F); }
            if (n >= 4) { ok = ok && ((b3 & 0xC0) == 0x80); cp = (cp << 6) | (b3 & 0x3F); }
            if (n == 3) ok = ok && cp >= 0x800 && !(cp >= 0xD800 && cp <= 0xDFFF);
            if (n == 4) ok = ok && cp >= 0x10000 && cp <= 0x10FFFF;
            u32 span = ((((1u << n) - 1) << (j + 3)) >> 3) & 0xFFFFu;   // bytes of this char inside the chunk
            if (!ok) { bad |= span; continue; }
            u32 c = tt_class_of(cp, T);
            u64 lane = (u64)span << ((c & 3) * 16);
            accA |= (c < 4) ? lane : 0ull;
            accB |= (c >= 4) ? lane : 0ull;
            cov |= span;
        }
        bad |= contm & ~cov;                                 // continuation byte without a lead
    }
    ChunkMasks m;
    m.lead = (u16)(lead & valid);
    m.oth = (u16)(accA & valid);          m.mark = (u16)((accA >> 16) & valid);
    m.spc = (u16)((accA >> 32) & valid);  m.num = (u16)((accA >> 48) & valid);
    m.low = (u16)(accB & valid);          m.upp = (u16)((accB >> 16) & valid);
    m.cless = (u16)((accB >> 32) & valid);
    m.nl = (u16)(accF & valid);           m.sp = (u16)((accF >> 16) & valid);
    m.ap = (u16)((accF >> 32) & valid);   m.sl = (u16)((accF >> 48) & valid);
    m.bad = (u16)(bad & valid);
    return m;
}

// Loads the chunk and its two 4-byte neighbours with aligned accesses and classifies it.
// `base` is 16-byte aligned; chunk in [0, nchunks); chunks outside that range are empty.
TT_HD ChunkMasks tt_classify_chunk(const u8* base, long long chunk, long long nchunks, long long lo, long long hi,
                                   const ClassTables& T) {
    u32 w[6] = {0, 0, 0, 0, 0, 0};
    if (chunk >= 0 && chunk < nchunks) {
        const uint4 v = *reinterpret_cast<const uint4*>(base + chunk * TT_CHUNK);
        w[1] = v.x; w[2] = v.y; w[3] = v.z; w[4] = v.w;
        if (chunk > 0) w[0] = *reinterpret_cast<const u32*>(base + chunk * TT_CHUNK - 4);
        if (chunk + 1 < nchunks) w[5] = *reinterpret_cast<const u32*>(base + (chunk + 1) * TT_CHUNK);
    }
    return tt_classify_words(w, chunk * TT_CHUNK, lo, hi, T);
}

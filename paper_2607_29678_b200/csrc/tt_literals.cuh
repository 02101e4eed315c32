// Added-token literal pass (paper Sec. 4.3 / 4.4): added and special tokens are literal strings that map to one
// reserved id each; a leftmost-longest pass extracts them before the tokenizer family handles the segments in
// between.  Two kernels prepare what the ordinary chain then consumes:
//   k_lit_scan    one thread per byte: the longest literal that matches at that byte (its length goes to
//                 cand[], its id to stage[] at the byte's text offset);
//   k_lit_select  leftmost-longest selection.  A candidate that no other candidate overlaps from the left is
//                 selected on its own; a chain of overlapping candidates is walked by the thread of its first
//                 member (each selected literal suppresses the candidates it covers, the next candidate behind
//                 it is selected in turn).  A selected literal becomes a document of its own in the boundary
//                 mask (so the segments around it are tokenized as independent texts), its first byte is
//                 marked in litstart and its other bytes in litin.
// k_pretok then forces exactly one piece per literal (start bit at its first byte, none inside) and, in its look-up
// half, takes the staged id for a piece that begins at a litstart bit.
#pragma once
#include "tt_common.cuh"

struct LitEntry { u32 first4; u32 off; u32 len; int32_t id; };       // first4: the first min(len, 4) bytes, low byte first
struct LitTable {
    const LitEntry* entries;     // sorted by length, longest first
    const u8* blob;              // the literals' bytes
    u32 n;
    u32 maxlen;
    u32 first_byte[8];           // bit b set: some literal begins with byte b
};

struct LitParams {
    const u8* base;              // aligned frame origin (text = base + lo)
    long long lo, hi;
    LitTable tab;
    u8* cand;                    // [hi + 1] aligned frame: length of the longest literal starting at the byte, 0 = none
    int32_t* stage;              // text offsets: id of that literal
    u32* docmask; u32* litstart; u32* litin;     // bit per byte, aligned frame (zero on entry)
};

__global__ void __launch_bounds__(256)
k_lit_scan(const LitParams P) {
    for (long long g = P.lo + (long long)blockIdx.x * blockDim.x + threadIdx.x; g < P.hi; g += (long long)gridDim.x * blockDim.x) {
        const u32 b = P.base[g];
        u32 found = 0;
        if ((P.tab.first_byte[b >> 5] >> (b & 31)) & 1) {
            const u32 avail = (u32)min((long long)P.tab.maxlen, P.hi - g);
            u32 w = b;
            for (u32 k = 1; k < 4 && k < avail; k++) w |= (u32)P.base[g + k] << (8 * k);
            for (u32 e = 0; e < P.tab.n && !found; e++) {          // longest first: the first match is the longest
                const LitEntry L = P.tab.entries[e];
                if (L.len > avail) continue;
                const u32 m = L.len >= 4 ? 0xFFFFFFFFu : (1u << (8 * L.len)) - 1;
                if ((w & m) != L.first4) continue;
                u32 k = 4;
                while (k < L.len && P.tab.blob[L.off + k] == P.base[g + k]) k++;
                if (k >= L.len) { found = L.len; P.stage[g - P.lo] = L.id; }
            }
        }
        P.cand[g] = (u8)found;
    }
}

__device__ __forceinline__ void lit_set_bits(u32* mask, long long from, long long to) {      // bits [from, to)
    while (from < to) {
        const long long wend = ((from >> 5) + 1) << 5, e = to < wend ? to : wend;
        const u32 bits = (e - from >= 32) ? 0xFFFFFFFFu : (((1u << (int)(e - from)) - 1) << (from & 31));
        atomicOr(&mask[from >> 5], bits);
        from = e;
    }
}

// Is some candidate q in (g - maxlen, g) long enough to cover byte g?
__device__ __forceinline__ bool lit_covered(const LitParams& P, long long g) {
    const long long lo = g - (long long)P.tab.maxlen + 1 > P.lo ? g - (long long)P.tab.maxlen + 1 : P.lo;
    for (long long q = g - 1; q >= lo; q--) {
        const u32 l = P.cand[q];
        if (l && q + l > g) return true;
    }
    return false;
}

__global__ void __launch_bounds__(256)
k_lit_select(const LitParams P) {
    if (blockIdx.x == 0 && threadIdx.x == 0) atomicOr(&P.docmask[P.lo >> 5], 1u << (P.lo & 31));      // the text itself starts a document
    for (long long g0 = P.lo + (long long)blockIdx.x * blockDim.x + threadIdx.x; g0 < P.hi; g0 += (long long)gridDim.x * blockDim.x) {
        if (!P.cand[g0] || lit_covered(P, g0)) continue;           // only the first member of a chain works
        long long g = g0;
        for (;;) {                                                 // bounded by the text length: g strictly grows
            const long long end = g + P.cand[g];
            lit_set_bits(P.litstart, g, g + 1);
            lit_set_bits(P.litin, g + 1, end);
            lit_set_bits(P.docmask, g, g + 1);
            if (end < P.hi) lit_set_bits(P.docmask, end, end + 1);
            // the next candidate at or behind `end`, if it belongs to this chain (something before it covers it)
            long long r = end;
            const long long stop = end + (long long)P.tab.maxlen < P.hi ? end + (long long)P.tab.maxlen : P.hi;
            while (r < stop && !P.cand[r]) r++;
            if (r >= stop || !lit_covered(P, r)) break;            // none near, or it heads a chain of its own
            g = r;
        }
    }
}

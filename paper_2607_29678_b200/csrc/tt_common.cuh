// Shared definitions of the toktier CUDA library (sm_100a).
#pragma once
#include <cstdint>
#include <cstddef>
#include <cuda_runtime.h>

#if defined(__CUDACC__)
#define TT_HD __host__ __device__ __forceinline__
// Rarely executed and large: kept out of line, so that the code a kernel runs through for every tile stays small
// enough for the instruction caches.
#define TT_HD_COLD __host__ __device__ __noinline__
#define TT_D_COLD __device__ __noinline__
#else
#define TT_HD inline
#define TT_HD_COLD inline
#endif

typedef uint8_t u8;
typedef uint16_t u16;
typedef uint32_t u32;
typedef uint64_t u64;

// ---- geometry of the pre-tokenization pass -------------------------------------------------
// A chunk is one aligned 16-byte vector load; a tile is what one CTA classifies per iteration.
constexpr int TT_CHUNK = 16;
#ifndef TT_TILE_CHUNKS_DEF
#define TT_TILE_CHUNKS_DEF 128
#endif
constexpr int TT_TILE_CHUNKS = TT_TILE_CHUNKS_DEF;        // = threads per CTA
constexpr int TT_TILE_BYTES = TT_CHUNK * TT_TILE_CHUNKS; // 2 KiB of text per tile
constexpr int TT_GROUP_TILES = 256;              // bulk text: token totals are also kept per group of 256 tiles
constexpr int TT_TILE_QCAP = TT_TILE_BYTES / 2;  // unsettled pieces of <= 256 bytes a tile can have (each has >= 2 bytes)
constexpr int TT_TILE_LONGCAP = 8;               // pieces of > 256 bytes that lie inside one tile
constexpr u32 TT_NONE = 0xFFFFFFFFu;

// ---- character class codes (two-stage Unicode table, see gen_unicode_table.py) ------------
enum : u32 { CC_OTHER = 0, CC_MARK = 1, CC_SPACE = 2, CC_NUMBER = 3, CC_LOWER = 4, CC_UPPER = 5, CC_CASELESS = 6 };

// ---- BPE -----------------------------------------------------------------------------------
constexpr u32 TT_ID_BITS = 18;                    // internal ids: byte b -> b, merge of rank r -> 256 + r
constexpr u32 TT_MAX_INTERNAL = 1u << TT_ID_BITS;
constexpr u32 TT_RANK_INF = 0xFFFFFFFFu;
constexpr u64 TT_SLOT_EMPTY = ~0ull;              // pair-table slot: (left << 38) | (right << 20) | rank
constexpr int TT_WARP_PIECE_MAX = 256;            // bytes; longer pieces take the block-cooperative path
// Bulk text: length classes of the pieces of at most 32 bytes (largest length of each class).
constexpr int TT_SHORT_CLASSES = 4;
TT_HD constexpr int tt_short_class_max(int c) { return c == 0 ? 10 : c == 1 ? 16 : c == 2 ? 22 : 32; }

// ---- workspace header (device memory) -----------------------------------------------------------
struct TTHeader {
    unsigned long long status_tag;   // (epoch of the call << 8) | device-side error code of that call
    u32 pretok_done;         // CTAs that finished the pre-tokenization pass (tt_pretokenize only; cleared by a memset)
    u32 n_pieces;            // number of pieces found (tt_pretokenize only)
    u32 t_tiles;             // ticket counter of k_merge's bulk mode (groups of tiles handed out); zeroed by the kernel before it
    u32 merge_done;          // CTAs of k_merge that have finished (bulk text: the last one sums the groups); zeroed likewise
    u32 nwq;                 // bulk text: lengths of the global lists of warp-class, short and long pieces and the ticket
    u32 nq_short, nq_long;   //            counter of the short list (all cleared by a memset before the chain)
    u32 t_short;
    u32 nq_short_x[3];       // bulk text: the short pieces have a list per length class; lengths of the other lists (cleared likewise)
    u32 dbg[8];              // first failed self-check of a kernel: site, then up to seven values (diagnostics only)
    u32 pad[11];
};
static_assert(sizeof(TTHeader) == 128, "header layout");

// The status word carries the epoch of the call that wrote it (a process-wide counter, never zero), so a
// value left by an earlier call -- or whatever an unused workspace holds -- reads as TT_OK and a single
// request needs no clearing pass before its first kernel.
#if defined(__CUDACC__)
// A kernel that finds one of its own indices out of range records where and what (first record wins), reports
// TT_ERR_INTERNAL_TIMEOUT through the status word and skips the access.
__device__ __forceinline__ void hdr_set_status(TTHeader* h, unsigned long long epoch, int code);
__device__ __noinline__ void hdr_selfcheck_failed(TTHeader* h, unsigned long long epoch, u32 site, u32 v0, u32 v1, u32 v2, u32 v3) {
    if (atomicCAS(&h->dbg[0], 0u, site) == 0u) { h->dbg[1] = v0; h->dbg[2] = v1; h->dbg[3] = v2; h->dbg[4] = v3; }
    hdr_set_status(h, epoch, 6 /* TT_ERR_INTERNAL_TIMEOUT */);
}
__device__ __forceinline__ int hdr_status(const TTHeader* h, unsigned long long epoch) {
    const unsigned long long t = *reinterpret_cast<const volatile unsigned long long*>(&h->status_tag);
    return (t >> 8) == epoch ? (int)(t & 0xFF) : 0;
}
__device__ __forceinline__ void hdr_set_status(TTHeader* h, unsigned long long epoch, int code) {   // the larger code stays
    unsigned long long old = *reinterpret_cast<volatile unsigned long long*>(&h->status_tag);
    for (int tries = 0; tries < 64; tries++) {
        const int cur = (old >> 8) == epoch ? (int)(old & 0xFF) : 0;
        if (cur >= code) return;
        const unsigned long long prev = atomicCAS(&h->status_tag, old, (epoch << 8) | (unsigned long long)code);
        if (prev == old) return;
        old = prev;
    }
}
#endif

// Per-tile records of the encode chain (all indexed by tile; a tile is TT_TILE_BYTES of the aligned frame).
// Nothing here is a global counter: every array element has exactly one writer in the first kernel, so that
// kernel needs neither atomics on global memory nor a clearing pass, and the layout does not depend on the
// order in which CTAs run.
//   tile_cnt[t]    pieces that start in the tile
//   tile_first[t]  offset in the tile of its first piece start, TT_NONE if it has none
//   tile_last[t]   offset in the tile of its last piece start (that piece ends in a later tile, or with the text)
//   tile_tok[t]    tokens of the tile's pieces (the first kernel stores the settled ones, k_merge adds the rest)
//   tile_q[t]      unsettled pieces: short (<= 32 B) count | warp-class (33..256 B) count << 11 | long count << 18
//   piece_off16    [t * TT_TILE_BYTES + i]  offset in the tile of piece i
//   piece_cnt      [t * TT_TILE_BYTES + i]  the id of piece i if it is one token found without merging (>= 0),
//                                           else minus the number of ids staged at the piece's text offset
//   q              [t * TT_TILE_QCAP ...]   queue entries of the tile: short pieces from the front, warp-class
//                                           pieces from the back; entry = offset in tile | index << 11 | (bytes-1) << 22
//   tile_long      [t * TT_TILE_LONGCAP + k] index of the k-th piece of > 256 bytes that lies inside the tile
struct TTWorkspace {
    TTHeader* hdr;
    u32* docmask;      // bit per text byte: first byte of a document (batch only)
    u16* startmask;    // bit per text byte: first byte of a piece, one u16 per chunk (tt_pretokenize and the cut pass only)
    u32* tile_cnt;     // (tt_pretokenize: then the exclusive prefix, ntiles + 1)
    u32* tile_first;
    u32* tile_last;
    u32* tile_tok;
    u32* tile_q;
    u32* grp_tok;      // bulk text only: tokens per group of TT_GROUP_TILES tiles
    u16* tile_long;
    u16* piece_off16;
    u32* piece_cnt;
    u32* q;
    u64* wq;           // bulk text only: warp-class pieces of all tiles (len / 33 + 64 entries)
    u64* gq;           // bulk text only: short pieces of all tiles by length class (see tt_short_class_max): a warp merges 32
    u64* gq_x[3];      // pieces of one list at a time, a thread each, and is done when the longest of them is
    uint4* lq;         // bulk text only: long pieces of all tiles (len / 257 + 16 entries)
    int32_t* stage;    // token ids staged at the byte offset of their piece (len)
    u64* pairbuf;      // (token, rank) pairs of the long-piece path, indexed like the text (len)
    u8* cand;          // literal pass: length of the longest added-token literal starting at each byte (aligned frame)
    u32* litstart;     // literal pass: bit per byte, first byte of an extracted literal
    u32* litin;        // literal pass: bit per byte, the other bytes of an extracted literal
    u32* cutmask;      // three-splitter composition: bit per byte, span starts of the first two stages
};

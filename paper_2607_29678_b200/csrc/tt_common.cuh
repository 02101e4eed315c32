// Shared definitions of the toktier CUDA library (sm_100a).
#pragma once
#include <cstdint>
#include <cstddef>
#include <cuda_runtime.h>

#if defined(__CUDACC__)
#define TT_HD __host__ __device__ __forceinline__
#else
#define TT_HD inline
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
constexpr int TT_GROUP_SHIFT = 8;                 // token totals are also kept per group of 256 tiles
constexpr int TT_GROUP_TILES = 1 << TT_GROUP_SHIFT;

// ---- character class codes (two-stage Unicode table, see gen_unicode_table.py) ------------
enum : u32 { CC_OTHER = 0, CC_MARK = 1, CC_SPACE = 2, CC_NUMBER = 3, CC_LOWER = 4, CC_UPPER = 5, CC_CASELESS = 6 };

// ---- BPE -----------------------------------------------------------------------------------
constexpr u32 TT_ID_BITS = 18;                    // internal ids: byte b -> b, merge of rank r -> 256 + r
constexpr u32 TT_MAX_INTERNAL = 1u << TT_ID_BITS;
constexpr u32 TT_RANK_INF = 0xFFFFFFFFu;
constexpr u64 TT_SLOT_EMPTY = ~0ull;              // pair-table slot: (left << 38) | (right << 20) | rank
constexpr int TT_WARP_PIECE_MAX = 256;            // bytes; longer pieces take the block-cooperative path

// ---- workspace header (device memory; counters zeroed by the call's first kernel or a memset) ----
struct TTHeader {
    unsigned long long status_tag;   // (epoch of the call << 8) | device-side error code of that call
    u32 pretok_done;         // CTAs that finished the pre-tokenization pass (tt_pretokenize only)
    u32 n_pieces;            // number of pieces found (tt_pretokenize only)
    u32 nq_short, nq_warp, nq_long;   // lengths of the queues of unsettled pieces (k_lookup)
    u32 t_short, t_warp;     // tickets of k_merge: queue entries handed out beyond the ones that warps own by index
    u32 pad[23];
};
static_assert(sizeof(TTHeader) == 128, "header layout");

// The status word carries the epoch of the call that wrote it (a process-wide counter, never zero), so a
// value left by an earlier call -- or whatever an unused workspace holds -- reads as TT_OK and a single
// request needs no clearing pass before its first kernel.
#if defined(__CUDACC__)
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

struct TTWorkspace {
    TTHeader* hdr;
    u32* docmask;      // bit per text byte: first byte of a document (batch only)
    u16* startmask;    // bit per text byte: first byte of a piece (one u16 per chunk)
    u32* tile_cnt;     // pieces per tile, then exclusive prefix (ntiles + 1)
    u32* tile_first;   // offset of the first piece start inside each tile, ~0 if none (ntiles + 1)
    u32* tile_tok;     // tokens per tile (ntiles + 1)
    u32* grp_tok;      // tokens per group of TT_GROUP_TILES tiles
    u32* piece_cnt;    // per piece, at tile * TT_TILE_BYTES + index inside the tile: its id (one token, no merging)
                       // or minus the staged token count
    int32_t* stage;    // token ids staged at the byte offset of their piece (len)
    u64* pairbuf;      // (token, rank) pairs of the long-piece path, indexed like the text (len)
    u64* q_short;      // unsettled pieces of <= 32 bytes (len / 2 + 64 entries)
    u64* q_warp;       // unsettled pieces of 33..256 bytes (len / 33 + 64 entries)
    uint4* q_long;     // unsettled longer pieces (len / 257 + 16 entries)
    u8* cand;          // literal pass: length of the longest added-token literal starting at each byte (aligned frame)
    u32* litstart;     // literal pass: bit per byte, first byte of an extracted literal
    u32* litin;        // literal pass: bit per byte, the other bytes of an extracted literal
    u32* cutmask;      // three-splitter composition: bit per byte, span starts of the first two stages
};

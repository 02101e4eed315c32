// Kernels of the pre-tokenization half: document mask, tag + piece-start flags (K1 + K2) with the
// per-tile piece counts and their prefix, and compaction into piece offsets (K3).
#pragma once
#include "tt_pretok.cuh"
#include "tt_pretok_p1.cuh"
#include "tt_bpe.cuh"

// ---- CTA-wide reductions over 256 threads (results broadcast to every thread) ---------------
__device__ __forceinline__ long long cta_max_ll(long long v, long long* scratch /* >= 9 */) {
    for (int o = 16; o; o >>= 1) { long long t = __shfl_xor_sync(0xFFFFFFFFu, v, o); v = t > v ? t : v; }
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    long long r = scratch[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); w++) r = scratch[w] > r ? scratch[w] : r;
    return r;
}
__device__ __forceinline__ u32 cta_sum_u32(u32 v, long long* scratch) {
    for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    u32 r = 0;
    for (int w = 0; w < (int)(blockDim.x >> 5); w++) r += (u32)scratch[w];
    return r;
}
// exclusive prefix of v over the CTA; *total receives the CTA sum
__device__ __forceinline__ u32 cta_exscan_u32(u32 v, u32* scratch /* >= 33 */, u32* total) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    u32 x = v;
    for (int o = 1; o < 32; o <<= 1) { u32 t = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += t; }
    __syncthreads();
    if (lane == 31) scratch[wid] = x;
    __syncthreads();
    if (wid == 0) {
        u32 s = lane < nw ? scratch[lane] : 0, y = s;
        for (int o = 1; o < 32; o <<= 1) { u32 t = __shfl_up_sync(0xFFFFFFFFu, y, o); if (lane >= o) y += t; }
        if (lane < nw) scratch[lane] = y - s;
        if (lane == nw - 1) scratch[32] = y;
    }
    __syncthreads();
    if (total) *total = scratch[32];
    return scratch[wid] + x - v;
}

// ---- document mask ---------------------------------------------------------------------------
// Sets the bit of every document's first byte (aligned frame).  Offsets must be ascending, start at
// 0 and end at the total length; a violation is reported as TT_ERR_ARG in the status word.
__global__ void k_docmask(const long long* __restrict__ doc_off, int n_docs, long long shift, long long len,
                          u32* __restrict__ docmask, TTHeader* hdr, unsigned long long epoch) {
    int d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d > n_docs) return;
    long long o = doc_off[d];
    bool ok = o >= 0 && o <= len && (d == 0 ? o == 0 : o >= doc_off[d - 1]) && (d < n_docs || o == len);
    if (!ok) { hdr_set_status(hdr, epoch, 1 /* TT_ERR_ARG */); return; }
    if (d < n_docs && o < len) {
        long long g = o + shift;
        atomicOr(&docmask[g >> 5], 1u << (g & 31));
    }
}

__device__ __forceinline__ u32 doc_bits(const PretokParams& P, long long chunk) {
    if (chunk < 0 || chunk >= P.nchunks) return 0;
    if (P.docmask) return reinterpret_cast<const u16*>(P.docmask)[chunk];
    return (chunk == (P.lo >> 4)) ? (1u << (P.lo & 15)) : 0u;
}

// ---- bounded CTA-cooperative walks over the text (runs that leave the shared-memory window) ----
// Every loop below advances by one tile per iteration and stops at the ends of the text.  All
// positions are in the aligned frame; `gend` is exclusive.

enum { RUN_NUM = 0, RUN_NL = 1, RUN_SL = 2 };
// The walks are rarely executed, so their instructions come from L2 or beyond, a cache line at a time: what a walk
// costs is mostly the size of the code it runs through.  They share one copy of the classifier.
TT_D_COLD ChunkMasks coop_classify(const PretokParams& P, const ClassTables& T, long long chunk) {
    return tt_classify_chunk(P.src ? P.src : P.base, chunk, P.nchunks, P.lo, P.hi, T);
}
constexpr long long COOP_NONE = -(1ll << 60);

__device__ __forceinline__ u32 run_mask(const ChunkMasks& m, int kind) {
    return kind == RUN_NUM ? m.num : kind == RUN_NL ? m.nl : m.sl;
}

// Walks down from gend-1 through bytes of the run class `kind` (cut at document starts).  Returns the
// position of the first byte that is not part of the run, with flags in the low three bits:
// 1 = the run was cut by a document start, 2 = that byte is "other" (4 = a mark), 8 = it is CR/LF.
// *leads receives the number of code-point leads inside the run (RUN_NUM only).
TT_D_COLD long long coop_back_run(const PretokParams& P, const ClassTables& T, long long gend, int kind,
                                   long long* scratch, u32* leads) {
    u32 total = 0;
    long long found = COOP_NONE;
    const long long ctop = (gend + TT_CHUNK - 1) / TT_CHUNK;          // chunks below ctop are examined
    for (long long cb = ctop - TT_TILE_CHUNKS;; cb -= TT_TILE_CHUNKS) {
        const long long chunk = cb + threadIdx.x;
        const ChunkMasks m = coop_classify(P, T, chunk);
        const u32 d = doc_bits(P, chunk), dn = doc_bits(P, chunk + 1);
        u32 live = 0xFFFFu;                                          // bytes of this chunk below gend
        if (chunk * 16 + 16 > gend) live = gend > chunk * 16 ? (0xFFFFu >> (int)(chunk * 16 + 16 - gend)) : 0u;
        const u32 dcut = ((d >> 1) | ((dn & 1) << 15));
        // a document start at gend itself does not cut the run (the caller has checked that byte)
        u32 dc = dcut;
        if (gend - 1 >= chunk * 16 && gend - 1 < chunk * 16 + 16) dc &= ~(1u << (int)(gend - 1 - chunk * 16));
        u32 cut = ((~run_mask(m, kind) & 0xFFFFu) | dc) & live;
        if (chunk < 0) cut = live;
        long long pos = COOP_NONE;
        if (cut) {
            const int b = tt_hibit(cut);
            const u32 flags = ((dc >> b) & 1) | ((((u32)m.oth >> b) & 1) << 1) | ((((u32)m.mark >> b) & 1) << 2) |
                              ((((u32)m.nl >> b) & 1) << 3);
            pos = ((chunk * 16 + b) << 4) | flags;
        }
        const long long top = cta_max_ll(pos, scratch);
        const long long top_pos = top == COOP_NONE ? COOP_NONE : (top >> 4);
        if (leads) {
            u32 mine = 0;
            if (chunk >= 0 && chunk * 16 + 15 > top_pos) {
                u32 keep = live;
                if (top_pos >= chunk * 16) keep &= (0xFFFFu << (int)(top_pos - chunk * 16 + 1));
                mine = tt_popc(m.lead & run_mask(m, kind) & keep);
            }
            total += cta_sum_u32(mine, scratch);
        }
        if (top != COOP_NONE) { found = top; break; }
        if (cb <= 0) { found = ((long long)-1 << 4) | 1; break; }
    }
    if (leads) *leads = total;
    return found;
}

// Number leads (mod 3) of the number run that ends right before gend.
TT_D_COLD u32 coop_back_num(const PretokParams& P, const ClassTables& T, long long gend, long long* scratch) {
    u32 leads = 0;
    coop_back_run(P, T, gend, RUN_NUM, scratch, &leads);
    return leads % 3;
}
// Is the byte before gend an "other" character, or a CR/LF run glued to one?  (marks count as
// "other" only for pattern 0)
TT_D_COLD u32 coop_back_nl(const PretokParams& P, const ClassTables& T, long long gend, long long* scratch) {
    const long long r = coop_back_run(P, T, gend, RUN_NL, scratch, nullptr);
    if (r & 1) return 0;
    return ((r >> 1) & 1) | (P.pattern != 1 ? ((r >> 2) & 1) : 0);
}
// Pattern 1: is the byte before gend a '/' run (or CR/LF run) that belongs to a punctuation tail?
TT_D_COLD u32 coop_back_slash(const PretokParams& P, const ClassTables& T, long long gend, long long* scratch) {
    const long long r = coop_back_run(P, T, gend, RUN_SL, scratch, nullptr);
    if ((r & 1) || !((r >> 3) & 1)) return 0;                 // cut by a document, or not preceded by CR/LF
    return coop_back_nl(P, T, (r >> 4) + 1, scratch);
}

// Does the whitespace run that continues at chunk c0 (its first byte) still contain a CR/LF?
TT_D_COLD u32 coop_fwd_nl(const PretokParams& P, const ClassTables& T, long long c0, long long* scratch) {
    for (long long cb = c0;; cb += TT_TILE_CHUNKS) {
        long long chunk = cb + threadIdx.x;
        ChunkMasks m = coop_classify(P, T, chunk);
        u32 d = doc_bits(P, chunk);
        u32 ev = ((~(u32)m.spc) | d | m.nl) & 0xFFFFu;       // bytes past the end are not whitespace
        long long neg = COOP_NONE;
        if (ev) {
            int j = tt_lobit(ev);
            u32 is_nl = ((u32)(m.nl & m.spc & ~d) >> j) & 1;
            // smallest position wins: negate, keep the answer in the low bit
            neg = -(((chunk * 16 + j) << 1) | (is_nl ^ 1));
        }
        long long best = cta_max_ll(neg, scratch);
        if (best != COOP_NONE) return (u32)(((-best) & 1) ^ 1);
        if (cb + TT_TILE_CHUNKS >= P.nchunks) return 0;
    }
}

// Pattern 1: nearest sure piece start (sure_only) or nearest sure-start / unresolved-construct event
// below gend.  Returns (position << 1) | is_unresolved; the text start is always a sure start.
TT_D_COLD long long coop_back_event(const PretokParams& P, const ClassTables& T, long long gend, bool sure_only,
                                     long long* scratch) {
    const long long ctop = (gend + TT_CHUNK - 1) / TT_CHUNK;
    for (long long cb = ctop - TT_TILE_CHUNKS;; cb -= TT_TILE_CHUNKS) {
        const long long chunk = cb + threadIdx.x;
        long long pos = COOP_NONE;
        if (chunk >= 0) {
            ChunkDoc p, c, n;
            p.m = coop_classify(P, T, chunk - 1); p.doc = doc_bits(P, chunk - 1);
            c.m = coop_classify(P, T, chunk);     c.doc = doc_bits(P, chunk);
            n.m = coop_classify(P, T, chunk + 1); n.doc = doc_bits(P, chunk + 1);
            tt_marks_inside_words_cm(p, c, n);
            u32 sure, hard;
            tt_sure_hard_cm(p, c, n, sure, hard);
            u32 live = 0xFFFFu;
            if (chunk * 16 + 16 > gend) live = gend > chunk * 16 ? (0xFFFFu >> (int)(chunk * 16 + 16 - gend)) : 0u;
            const u32 ev = (sure | (sure_only ? 0u : hard)) & live;
            if (ev) { const int b = tt_hibit(ev); pos = ((chunk * 16 + b) << 1) | (sure_only ? 0u : ((hard >> b) & 1)); }
        }
        const long long top = cta_max_ll(pos, scratch);
        if (top != COOP_NONE) return top;
        if (cb <= 0) return (P.lo << 1);
    }
}

// ---- K1 + K2 -----------------------------------------------------------------------------------
__device__ __forceinline__ void store_slot(u16 (*sm)[TT_SLOTS], int s, const ChunkMasks& m, u32 d) {
    sm[F_LEAD][s] = m.lead; sm[F_OTH][s] = m.oth; sm[F_MARK][s] = m.mark; sm[F_SPC][s] = m.spc;
    sm[F_NUM][s] = m.num; sm[F_LOW][s] = m.low; sm[F_UPP][s] = m.upp; sm[F_CLESS][s] = m.cless;
    sm[F_NL][s] = m.nl; sm[F_SP][s] = m.sp; sm[F_AP][s] = m.ap; sm[F_SL][s] = m.sl; sm[F_DOC][s] = (u16)d;
}

// What the fused kernel needs beyond the piece-start predicate: the per-tile records it leaves (see TTWorkspace)
// and the tables of the whole-piece lookups.
struct FrontParams {
    u32* tile_last; u32* tile_tok; u32* tile_q; u16* tile_long; u16* piece_off16; u32* piece_cnt; u32* q;
    u64* wq;                   // bulk text (more tiles than a request's job search covers): the warp-class pieces of all tiles go
                               // to this one list, appended tile by tile (hdr->nwq, cleared before the chain); else null
    TokTable toktab;           // slots == nullptr: none
    LongTable longtab;         // ignore_merges: entries longer than the whole-piece table holds (else slots == nullptr)
    const int32_t* ext_id;
};

// A piece on the general path of the fused kernel: an extracted literal, a single byte, a vocabulary entry of up to
// 24 bytes, or (ignore_merges) a longer entry.  Returns true and the value for piece_cnt if it needs no merging.
__device__ __forceinline__ bool front_piece_general(const PretokParams& P, const FrontParams& F, const u8* __restrict__ text, u32 a, u32 n, u32& val) {
    int32_t id;
    if (P.litstart != nullptr) {
        const long long g = (long long)a + P.lo;
        if ((P.litstart[g >> 5] >> (g & 31)) & 1) { val = 0u - 1u; return true; }    // one staged id (written by the literal pass)
    }
    if (n == 1) { val = (u32)F.ext_id[text[a]]; return true; }
    if (n <= (u32)TT_TOKTAB_MAXLEN) {
        if (F.toktab.slots != nullptr && toktab_lookup(F.toktab, text, a, n, id)) { val = (u32)id; return true; }
    } else if (F.longtab.slots != nullptr && n <= F.longtab.maxlen && longtab_lookup(F.longtab, text, a, n, id)) { val = (u32)id; return true; }
    return false;
}
// An unsettled piece (offset o in the tile, index i, n bytes) goes to the tile's queue of its length class.
__device__ __forceinline__ void front_piece_queue(const FrontParams& F, int tile, u32 o, u32 i, u32 n, u32* s_ns, u32* s_nw, u32* s_nl, u16* s_wlist) {
    if (n > (u32)TT_WARP_PIECE_MAX) F.tile_long[(size_t)tile * TT_TILE_LONGCAP + atomicAdd(s_nl, 1u)] = (u16)i;
    else if (n > (u32)LANE_MAX) {
        const u32 k = atomicAdd(s_nw, 1u);
        if (F.wq != nullptr) s_wlist[k] = (u16)i;
        else F.q[(size_t)tile * TT_TILE_QCAP + (u32)TT_TILE_QCAP - 1 - k] = tile_queue_entry(o, i, n);
    }
    else F.q[(size_t)tile * TT_TILE_QCAP + atomicAdd(s_ns, 1u)] = tile_queue_entry(o, i, n);
}

// FUSED = false: the start flags go to P.startmask, with the pieces per tile (tt_pretokenize and the cut pass of the
// three-splitter composition).
// FUSED = true (the encode chain's first kernel): the tile's flags stay in shared memory and become its list of
// piece offsets (K3); every piece but the tile's last one -- whose end another tile knows -- is settled here if it
// is a single byte, an extracted literal or a whole vocabulary entry (one 32-byte probe), and queued for k_merge
// otherwise.  Everything a tile leaves behind has this CTA as its only writer: no atomics on global memory, no
// counter that would have to be cleared before the call.
// MINB = CTAs per SM the kernel is compiled for.  A request (at most a few tiles per CTA) is a latency chain and
// gets the registers it wants (6 CTAs of 128 threads, 80 registers) and four table look-ups in flight per thread.
// Bulk text is bound by instruction issue and by the latencies between its barriers, which more resident warps
// hide better than anything a thread does for itself: 16 CTAs per SM (every warp slot taken, 32 registers, a few
// spills) with one look-up at a time per thread.  The 132 MB batch: 1.80 ms at 6 CTAs, 1.64 at 10, 1.42 with the
// rare paths out of line, 1.34 with one look-up in flight instead of four, 1.31 at 12 CTAs, 1.28 at 16.
constexpr int PRETOK_CTAS_REQUEST = 6, PRETOK_CTAS_BULK = 16;
// PAT = the pattern the kernel is compiled for (P.pattern says the same): each pattern's rules are a few hundred
// kilobytes of code, and a kernel that carries all of them keeps missing the instruction caches on its way through
// the one it runs.
template <bool FUSED, int MINB, int PAT>
__global__ void __launch_bounds__(TT_TILE_CHUNKS, MINB)
k_pretok(const __grid_constant__ PretokParams P, const __grid_constant__ FrontParams F) {
    extern __shared__ __align__(16) u8 smem_raw[];
    u16 (*sm)[TT_SLOTS] = reinterpret_cast<u16 (*)[TT_SLOTS]>(smem_raw);        // class masks of the tile and its halo
    u32* const s_runmask = reinterpret_cast<u32*>(smem_raw + TT_RUNMASK_OFFSET);   // run summaries of the slots, behind the masks
    // Only the kernel compiled for requests fills them (a request may be one long run; its tiles each get a CTA that
    // the others wait for).  Bulk text pays for every instruction per tile: there the summaries stay empty and the
    // walks visit slot after slot.
    constexpr bool RUN_SUMMARIES = MINB <= PRETOK_CTAS_REQUEST;
    if (!RUN_SUMMARIES && threadIdx.x < 2 * TT_RUNMASK_WORDS) s_runmask[threadIdx.x] = 0;     // (the first barrier of the tile loop orders this)
    __shared__ long long scratch[40];
    __shared__ u32 s_need, s_first;
    __shared__ u32 s_islast;
    __shared__ u16 s_off[FUSED ? TT_TILE_BYTES + 2 : 2];              // piece offsets of the tile
    __shared__ u32 s_wtot[TT_TILE_CHUNKS / 32], s_ns, s_nw, s_nl, s_total, s_wbase;
    __shared__ u16 s_wlist[TT_TILE_BYTES / (LANE_MAX + 1) + 2];       // bulk text: the tile's warp-class pieces
    __shared__ u16 s_slow[TT_TILE_BYTES / 9 + 4];                     // pieces of more than 8 bytes (looked up together)
    __shared__ u32 s_nslow;

    const int tid = threadIdx.x;
    cudaTriggerProgrammaticLaunchCompletion();               // the next kernel may be placed; it waits for this grid's memory itself
    if (FUSED) {
        if (blockIdx.x == 0 && tid == 0) { P.hdr->t_tiles = 0; P.hdr->merge_done = 0; }   // k_merge's counters (k_merge touches them only after this grid)
        // the whole-piece table is probed at random a few microseconds from now: ask for it to be brought into L2
        if (F.toktab.slots != nullptr) grid_prefetch_l2(F.toktab.slots, ((size_t)F.toktab.mask + 1) * sizeof(TokSlot));
    }
    // The class tables stay in global memory (21 KB, read through L1): chunks of plain ASCII -- nearly all of a
    // transcript -- are classified without any table, so shared memory is left to the masks and more CTAs fit an SM.
    ClassTables T;
    T.stage1 = P.cls_tables; T.stage2 = P.cls_tables + 0x1100; T.ascii = P.cls_tables + P.cls_bytes - 128;
    SeqCtx SC;
    // Where the text is read from: the device buffer, or (host calls with pinned text) the caller's host memory.  In
    // the second case the CTA that classifies a chunk also writes it to the device copy; this kernel reads that copy
    // only for the look-ups of the tile's own pieces, behind the tile's barriers.
    const u8* const rd = P.src ? P.src : P.base;
    SC.base = rd; SC.lo = P.lo; SC.hi = P.hi; SC.docmask = P.docmask; SC.T = T;
    u32 any_bad = 0;

    for (int tile = blockIdx.x; tile < P.ntiles; tile += gridDim.x) {
        __syncthreads();
        if (tid == 0) { s_need = 0; s_first = 0xFFFFFFFFu; s_ns = 0; s_nw = 0; s_nl = 0; s_total = 0; s_nslow = 0; }
        const long long c_first = (long long)tile * TT_TILE_CHUNKS;
        // phase A: classify own chunk (+ the halo chunks)
        {
            const long long chunk = c_first + tid;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (chunk < P.nchunks) {
                v = *reinterpret_cast<const uint4*>(rd + chunk * TT_CHUNK);
                if (P.src) *reinterpret_cast<uint4*>(P.copy + chunk * TT_CHUNK) = v;
            }
            const ChunkMasks m = tt_classify_chunk_loaded(v, rd, chunk, P.nchunks, P.lo, P.hi, T);
            const u32 d = doc_bits(P, chunk);
            store_slot(sm, tid + TT_LOW_HALO, m, d);
            any_bad |= m.bad | (d & ~(u32)m.lead & 0xFFFFu & (m.oth | m.mark | m.spc | m.num | m.low | m.upp | m.cless));
            if (RUN_SUMMARIES) {      // (see tt_runmask) is the slot sixteen ASCII digits / sixteen blanks other than CR/LF?
                const u32 bn = __ballot_sync(0xFFFFFFFFu, m.num == 0xFFFFu && m.lead == 0xFFFFu && d == 0);
                const u32 bb = __ballot_sync(0xFFFFFFFFu, m.spc == 0xFFFFu && m.nl == 0 && d == 0);
                if ((tid & 31) == 0) { s_runmask[tid >> 5] = bn; s_runmask[TT_RUNMASK_WORDS + (tid >> 5)] = bb; }
            }
        }
        if (tid < 32) {                                               // the halo slots: the first warp
            bool hn = false, hb = false;
            if (tid < TT_LOW_HALO + 1) {
                const long long chunk = tid < TT_LOW_HALO ? c_first - TT_LOW_HALO + tid : c_first + TT_TILE_CHUNKS;
                const int s = tid < TT_LOW_HALO ? tid : TT_SLOTS - 1;
                const ChunkMasks m = tt_classify_chunk(rd, chunk, P.nchunks, P.lo, P.hi, T);
                const u32 d = doc_bits(P, chunk);
                store_slot(sm, s, m, d);
                hn = m.num == 0xFFFFu && m.lead == 0xFFFFu && d == 0;
                hb = m.spc == 0xFFFFu && m.nl == 0 && d == 0;
            }
            if (RUN_SUMMARIES) {
                const u32 bn = __ballot_sync(0xFFFFFFFFu, hn), bb = __ballot_sync(0xFFFFFFFFu, hb);
                if (tid == 0) { s_runmask[TT_TILE_CHUNKS / 32] = bn | 0x80000000u; s_runmask[TT_RUNMASK_WORDS + TT_TILE_CHUNKS / 32] = bb | 0x80000000u; }
            }
        }
        __syncthreads();
        if (PAT == 1) {                                          // marks inside words count as caseless letters from here on
            const u32 in_own = tt_marks_inside_words(sm, tid + TT_LOW_HALO);
            const int hs = tid < TT_LOW_HALO ? tid : TT_SLOTS - 1;
            const u32 in_halo = tid < TT_LOW_HALO + 1 ? tt_marks_inside_words(sm, hs) : 0u;
            __syncthreads();
            if (in_own) { sm[F_MARK][tid + TT_LOW_HALO] &= (u16)~in_own; sm[F_CLESS][tid + TT_LOW_HALO] |= (u16)in_own; }
            if (in_halo) { sm[F_MARK][hs] &= (u16)~in_halo; sm[F_CLESS][hs] |= (u16)in_halo; }
            __syncthreads();
        }
        if (PAT == 1) {                                          // sure starts / unresolved constructs per slot
            u32 su, ha;
            const long long gs0 = (c_first - TT_LOW_HALO) * TT_CHUNK;       // byte 0 of slot 0
            tt_sure_hard(sm, tid + TT_LOW_HALO, su, ha, rd, gs0, P.hi);
            sm[F_SURE][tid + TT_LOW_HALO] = (u16)su; sm[F_HARD][tid + TT_LOW_HALO] = (u16)ha;
            if (tid >= 1 && tid < TT_LOW_HALO) { tt_sure_hard(sm, tid, su, ha, rd, gs0, P.hi); sm[F_SURE][tid] = (u16)su; sm[F_HARD][tid] = (u16)ha; }
            __syncthreads();
        }
        // phase B: evaluate the piece-start predicate
        TileCarry tc;
        tc.n_before = 0; tc.nl_absorbed_before = 0; tc.nl_later_after = 0; tc.slash_absorbed_before = 0;
        tc.dirty_before = 0; tc.sure_before = P.lo;
        u32 need = 0;
        const int slot = tid + TT_LOW_HALO;
        const long long g0 = (c_first + tid) * TT_CHUNK;
        u32 S = PAT == TT_PATTERN_CUTS ? tt_eval_chunk_cuts(sm, slot, tc, false, need)
              : PAT != 1 ? tt_eval_chunk_p0(sm, slot, rd, g0, P.hi, tc, false, need, PAT == 2, P.docmask)
                         : tt_eval_chunk_p1(sm, slot, SC, g0, tc, false, need);
        if (need) atomicOr(&s_need, need);
        __syncthreads();
        const u32 need_all = s_need;
        if (need_all) {                                               // block-uniform
            const long long below = (c_first - TT_LOW_HALO) * TT_CHUNK;    // first byte of the low halo
            if (need_all & NEED_N) tc.n_before = coop_back_num(P, T, below, scratch);
            if (need_all & NEED_A) tc.nl_absorbed_before = coop_back_nl(P, T, below, scratch);
            if (PAT == 1 && (need_all & NEED_S)) tc.slash_absorbed_before = coop_back_slash(P, T, below, scratch);
            if (need_all & NEED_F) tc.nl_later_after = coop_fwd_nl(P, T, c_first + TT_TILE_CHUNKS + 1, scratch);
            if (PAT == 1 && (need_all & (NEED_H | NEED_C))) {
                // events of slot 0 (first halo chunk) are not examined by the walks in shared memory
                const long long gend = below + TT_CHUNK;
                const long long ev = coop_back_event(P, T, gend, false, scratch);
                tc.dirty_before = (u32)(ev & 1);
                tc.sure_before = (ev & 1) ? (coop_back_event(P, T, (ev >> 1) + 1, true, scratch) >> 1) : (ev >> 1);
            }
            need = 0;
            S = PAT == TT_PATTERN_CUTS ? tt_eval_chunk_cuts(sm, slot, tc, true, need)
              : PAT != 1 ? tt_eval_chunk_p0(sm, slot, rd, g0, P.hi, tc, true, need, PAT == 2, P.docmask)
                         : tt_eval_chunk_p1(sm, slot, SC, g0, tc, true, need);
        }
        if (P.litstart && c_first + tid < P.nchunks) {                // an extracted literal is one piece whatever the pattern says
            const long long chunk = c_first + tid;
            S = (S & ~(u32)reinterpret_cast<const u16*>(P.litin)[chunk]) | reinterpret_cast<const u16*>(P.litstart)[chunk];
        }
        if (!FUSED) {
            if (c_first + tid < P.nchunks) P.startmask[c_first + tid] = (u16)S;
            if (S) atomicMin(&s_first, (u32)(tid * TT_CHUNK + tt_lobit(S)));
            u32 total = cta_sum_u32(tt_popc(S), scratch);
            if (tid == 0) { P.tile_cnt[tile] = total; P.tile_first[tile] = s_first; }
            continue;
        }
        // ---- K3 in shared memory: the tile's piece offsets ------------------------------------------------------
        const int lane = tid & 31, wid = tid >> 5;
        const u32 cnt = tt_popc(S);
        u32 x = cnt;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) { const u32 t = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += t; }
        if (lane == 31) s_wtot[wid] = x;
        __syncthreads();
        u32 np = 0, r = x - cnt;
#pragma unroll
        for (int w = 0; w < TT_TILE_CHUNKS / 32; w++) { const u32 v = s_wtot[w]; np += v; if (w < wid) r += v; }
        for (u32 m = S; m; m &= m - 1) s_off[r++] = (u16)(tid * TT_CHUNK + tt_lobit(m));
        __syncthreads();
        const size_t p0 = (size_t)tile * TT_TILE_BYTES;              // pieces are indexed per tile
        for (u32 i = tid; i < np; i += TT_TILE_CHUNKS) F.piece_off16[p0 + i] = s_off[i];
        if (tid == 0) {
            P.tile_cnt[tile] = np;
            P.tile_first[tile] = np ? (u32)s_off[0] : TT_NONE;
            F.tile_last[tile] = np ? (u32)s_off[np - 1] : TT_NONE;
        }
        // ---- K4, first half: whole-piece lookups, a thread per piece, four pieces per thread and step, their loads side
        // by side (a lookup is a chain of two dependent loads: the text words, then the table slot).  Pieces of at most 8
        // bytes -- most of them -- take a path of their own: two key words, one 16-byte half of the slot.  The tile's last
        // piece is left to k_merge.
        const u8* text = P.base + P.lo;
        const long long t0 = c_first * TT_CHUNK - P.lo;               // text offset of the tile start
        const u32 nlook = np ? np - 1 : 0;
        const bool quick = P.litstart == nullptr && F.toktab.slots != nullptr;     // block-uniform
        u32 wsum = 0;
        constexpr int LW = MINB > PRETOK_CTAS_REQUEST ? 1 : 4;       // look-ups in flight per thread
        for (u32 ib = tid; ib < nlook; ib += LW * TT_TILE_CHUNKS) {
            u32 o[LW], n[LW], k0[LW], k1[LW], h[LW], x0[LW], x1[LW], x2[LW];
            uint4 sl[LW];
#pragma unroll
            for (int j = 0; j < LW; j++) {
                const u32 i = ib + j * TT_TILE_CHUNKS;
                o[j] = 0; n[j] = 0; x0[j] = 0; x1[j] = 0; x2[j] = 0;
                if (i < nlook) { o[j] = s_off[i]; n[j] = (u32)s_off[i + 1] - o[j]; }
                if (quick && n[j] != 0 && n[j] <= 8) {
                    const uintptr_t addr = (uintptr_t)(text + t0 + o[j]);
                    const u32* w = reinterpret_cast<const u32*>(addr & ~(uintptr_t)3);
                    const u32 used = (u32)(addr & 3) + n[j];
                    x0[j] = w[0];                                         // (plain loads: this CTA may have written these bytes itself)
                    if (used > 4) x1[j] = w[1];
                    if (used > 8) x2[j] = w[2];
                }
            }
#pragma unroll
            for (int j = 0; j < LW; j++) {
                k0[j] = 0; k1[j] = 0; h[j] = 0; sl[j] = make_uint4(0, 0, 0, 0);
                if (quick && n[j] != 0 && n[j] <= 8) {
                    toktab_key01(x0[j], x1[j], x2[j], (u32)((uintptr_t)(text + t0 + o[j]) & 3), n[j], k0[j], k1[j]);
                    if (n[j] == 1) sl[j].y = (u32)F.ext_id[k0[j]];
                    else {
                        h[j] = toktab_hash_final(toktab_hash_short(k0[j], k1[j], n[j]), F.toktab.shift);
                        sl[j] = __ldg(reinterpret_cast<const uint4*>(F.toktab.slots + h[j]));
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < LW; j++) {
                const u32 i = ib + j * TT_TILE_CHUNKS;
                if (n[j] == 0) continue;
                bool settled = false;
                u32 val = 0;
                if (quick && n[j] == 1) { val = sl[j].y; settled = true; }
                else if (quick && n[j] <= 8) {
                    uint4 c = sl[j];
                    u32 hh = h[j];
                    for (u32 probe = 0; probe <= F.toktab.mask; probe++) {       // bounded by the capacity
                        if (c.x == 0) break;
                        if (c.x == n[j] && c.z == k0[j] && c.w == k1[j]) { val = c.y; settled = true; break; }
                        hh = (hh + 1) & F.toktab.mask;
                        c = __ldg(reinterpret_cast<const uint4*>(F.toktab.slots + hh));
                    }
                } else if (quick) { s_slow[atomicAdd(&s_nslow, 1u)] = (u16)i; continue; }     // longer pieces: together, below
                else settled = front_piece_general(P, F, text, (u32)(t0 + o[j]), n[j], val);
                if (settled) { F.piece_cnt[p0 + i] = val; wsum++; }
                else front_piece_queue(F, tile, o[j], i, n[j], &s_ns, &s_nw, &s_nl, s_wlist);
            }
        }
        if (quick) {                                                  // block-uniform: the pieces of more than 8 bytes, a thread each
            __syncthreads();
            const u32 nslow = s_nslow;
            for (u32 e = tid; e < nslow; e += TT_TILE_CHUNKS) {
                const u32 i = s_slow[e], o = s_off[i], n = (u32)s_off[i + 1] - o;
                u32 val = 0;
                if (front_piece_general(P, F, text, (u32)(t0 + o), n, val)) { F.piece_cnt[p0 + i] = val; wsum++; }
                else front_piece_queue(F, tile, o, i, n, &s_ns, &s_nw, &s_nl, s_wlist);
            }
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) wsum += __shfl_xor_sync(0xFFFFFFFFu, wsum, o);
        if (lane == 0 && wsum) atomicAdd(&s_total, wsum);
        __syncthreads();
        if (tid == 0) {
            F.tile_tok[tile] = s_total;
            F.tile_q[tile] = s_ns | ((F.wq != nullptr ? 0u : s_nw) << TQ_NW_SHIFT) | (s_nl << TQ_NL_SHIFT);
            if (F.wq != nullptr && s_nw) s_wbase = atomicAdd(&P.hdr->nwq, s_nw);
        }
        if (F.wq != nullptr && s_nw) {                                // block-uniform
            __syncthreads();
            for (u32 k = tid; k < s_nw; k += TT_TILE_CHUNKS) {
                const u32 i = s_wlist[k];
                F.wq[s_wbase + k] = ((u64)(u32)tile << 32) | tile_queue_entry(s_off[i], i, (u32)s_off[i + 1] - s_off[i]);
            }
        }
    }
    if (any_bad) hdr_set_status(P.hdr, P.epoch, 4 /* TT_ERR_INVALID_UTF8 */);

    // the last CTA to finish turns the tile counts into their exclusive prefix (only where the piece list is
    // materialised: the encode chain indexes its pieces per tile and needs no prefix)
    if (FUSED || !P.want_prefix) return;
    __threadfence();
    __syncthreads();
    if (tid == 0) s_islast = (atomicAdd(&P.hdr->pretok_done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (s_islast) {
        __threadfence();
        u32* sc = reinterpret_cast<u32*>(scratch);
        u32 carry = 0;
        for (int b0 = 0; b0 < P.ntiles; b0 += blockDim.x) {
            int i = b0 + tid;
            u32 v = i < P.ntiles ? P.tile_cnt[i] : 0, tot;
            u32 ex = cta_exscan_u32(v, sc, &tot);
            if (i < P.ntiles) P.tile_cnt[i] = carry + ex;
            carry += tot;
            __syncthreads();
        }
        if (tid == 0) { P.tile_cnt[P.ntiles] = carry; P.hdr->n_pieces = carry; }
    }
}

// ---- K3: compaction of the start flags into piece offsets (tt_pretokenize) --------------------------
// piece_off[i] = byte offset (relative to the text) of piece i; piece_off[n_pieces] = len.  The encode
// chain does the same per tile in shared memory (the fused half of k_pretok) and keeps the offsets per tile.
__global__ void __launch_bounds__(TT_TILE_CHUNKS)
k_compact(const u16* __restrict__ startmask, const u32* __restrict__ tile_base, long long nchunks, int ntiles,
          long long shift, long long len, u32* __restrict__ piece_off, TTHeader* hdr, unsigned long long epoch) {
    __shared__ u32 sc[40];
    if (hdr_status(hdr, epoch) != 0) return;
    for (int tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const long long chunk = (long long)tile * TT_TILE_CHUNKS + threadIdx.x;
        u32 m = chunk < nchunks ? startmask[chunk] : 0;
        u32 r = tile_base[tile] + cta_exscan_u32(tt_popc(m), sc, nullptr);
        const long long g0 = chunk * TT_CHUNK - shift;
        while (m) { int i = tt_lobit(m); m &= m - 1; piece_off[r++] = (u32)(g0 + i); }
        __syncthreads();
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) piece_off[tile_base[ntiles]] = (u32)len;
}

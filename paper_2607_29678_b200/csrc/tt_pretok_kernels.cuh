// Kernels of the pre-tokenization half: document mask, tag + piece-start flags (K1 + K2) with the
// per-tile piece counts and their prefix, and compaction into piece offsets (K3).
#pragma once
#include "tt_pretok.cuh"
#include "tt_pretok_p1.cuh"

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
                          u32* __restrict__ docmask, TTHeader* hdr) {
    int d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d > n_docs) return;
    long long o = doc_off[d];
    bool ok = o >= 0 && o <= len && (d == 0 ? o == 0 : o >= doc_off[d - 1]) && (d < n_docs || o == len);
    if (!ok) { atomicMax(&hdr->status, 1 /* TT_ERR_ARG */); return; }
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
// Every loop below advances by one tile per iteration and stops at the ends of the text.

// Number leads (mod 3) of the number run that ends right before chunk c0.
__device__ u32 coop_back_num(const PretokParams& P, const ClassTables& T, long long c0, long long* scratch) {
    u32 total = 0;
    for (long long cb = c0 - TT_TILE_CHUNKS;; cb -= TT_TILE_CHUNKS) {
        long long chunk = cb + threadIdx.x;
        ChunkMasks m = tt_classify_chunk(P.base, chunk, P.nchunks, P.lo, P.hi, T);
        u32 d = doc_bits(P, chunk), dn = doc_bits(P, chunk + 1);
        u32 cut = (~(u32)m.num & 0xFFFFu) | (d >> 1) | ((dn & 1) << 15);
        if (chunk < 0) cut = 0xFFFFu;
        long long pos = cut ? chunk * 16 + tt_hibit(cut) : -(1ll << 60);
        long long top = cta_max_ll(pos, scratch);
        u32 mine = 0;
        if (chunk * 16 + 15 > top) {
            u32 keep = 0xFFFFu;
            if (top >= chunk * 16) keep = (0xFFFFu << (int)(top - chunk * 16 + 1)) & 0xFFFFu;
            mine = tt_popc(m.lead & m.num & keep);
        }
        total += cta_sum_u32(mine, scratch);
        if (top > -(1ll << 59) || cb <= 0) break;
    }
    return total % 3;
}

// Is the CR/LF run that ends right before chunk c0 glued to a preceding punctuation character?
__device__ u32 coop_back_nl(const PretokParams& P, const ClassTables& T, long long c0, long long* scratch) {
    for (long long cb = c0 - TT_TILE_CHUNKS;; cb -= TT_TILE_CHUNKS) {
        long long chunk = cb + threadIdx.x;
        ChunkMasks m = tt_classify_chunk(P.base, chunk, P.nchunks, P.lo, P.hi, T);
        u32 d = doc_bits(P, chunk), dn = doc_bits(P, chunk + 1);
        u32 dcut = (d >> 1) | ((dn & 1) << 15);
        u32 cut = (~(u32)m.nl & 0xFFFFu) | dcut;
        if (chunk < 0) cut = 0xFFFFu;
        long long pos = -(1ll << 60);
        if (cut) {
            int b = tt_hibit(cut);
            // encode the answer in the low bit: (position << 1) | glued
            u32 glued = (chunk >= 0) && !((dcut >> b) & 1) && (((u32)(m.oth | m.mark) >> b) & 1);
            pos = ((chunk * 16 + b) << 1) | glued;
        }
        long long top = cta_max_ll(pos, scratch);
        if (top > -(1ll << 59)) return (u32)(top & 1);
        if (cb <= 0) return 0;
    }
}

// Does the whitespace run that continues at chunk c0 (its first byte) still contain a CR/LF?
__device__ u32 coop_fwd_nl(const PretokParams& P, const ClassTables& T, long long c0, long long* scratch) {
    for (long long cb = c0;; cb += TT_TILE_CHUNKS) {
        long long chunk = cb + threadIdx.x;
        ChunkMasks m = tt_classify_chunk(P.base, chunk, P.nchunks, P.lo, P.hi, T);
        u32 d = doc_bits(P, chunk);
        u32 ev = ((~(u32)m.spc) | d | m.nl) & 0xFFFFu;       // bytes past the end are not whitespace
        long long neg = -(1ll << 60);
        if (ev) {
            int j = tt_lobit(ev);
            u32 is_nl = ((u32)(m.nl & m.spc & ~d) >> j) & 1;
            // smallest position wins: negate, keep the answer in the low bit
            neg = -(((chunk * 16 + j) << 1) | (is_nl ^ 1));
        }
        long long best = cta_max_ll(neg, scratch);
        if (best > -(1ll << 59)) return (u32)(((-best) & 1) ^ 1);
        if (cb + TT_TILE_CHUNKS >= P.nchunks) return 0;
    }
}

// ---- K1 + K2 -----------------------------------------------------------------------------------
__global__ void __launch_bounds__(TT_TILE_CHUNKS)
k_pretok(const PretokParams P) {
    extern __shared__ __align__(16) u8 smem_raw[];
    u8* tables = smem_raw;                                            // class tables
    u16 (*sm)[TT_SLOTS] = reinterpret_cast<u16 (*)[TT_SLOTS]>(smem_raw + ((P.cls_bytes + 15) & ~15));
    __shared__ long long scratch[40];
    __shared__ u32 s_need;
    __shared__ TileCarry s_tc;
    __shared__ u32 s_islast;

    const int tid = threadIdx.x;
    for (int i = tid * 16; i < P.cls_bytes; i += blockDim.x * 16)
        *reinterpret_cast<uint4*>(tables + i) = *reinterpret_cast<const uint4*>(P.cls_tables + i);
    ClassTables T;
    T.stage1 = tables; T.stage2 = tables + 0x1100; T.ascii = tables + P.cls_bytes - 128;
    u32 any_bad = 0;

    for (int tile = blockIdx.x; tile < P.ntiles; tile += gridDim.x) {
        __syncthreads();
        if (tid == 0) s_need = 0;
        const long long c_first = (long long)tile * TT_TILE_CHUNKS;
        // phase A: classify own chunk (+ the two halo chunks)
        {
            const long long chunk = c_first + tid;
            ChunkMasks m = tt_classify_chunk(P.base, chunk, P.nchunks, P.lo, P.hi, T);
            const int s = tid + 1;
            u32 d = doc_bits(P, chunk);
            sm[F_LEAD][s] = m.lead; sm[F_OTH][s] = m.oth; sm[F_MARK][s] = m.mark; sm[F_SPC][s] = m.spc;
            sm[F_NUM][s] = m.num; sm[F_LOW][s] = m.low; sm[F_UPP][s] = m.upp; sm[F_CLESS][s] = m.cless;
            sm[F_NL][s] = m.nl; sm[F_SP][s] = m.sp; sm[F_AP][s] = m.ap; sm[F_SL][s] = m.sl; sm[F_DOC][s] = (u16)d;
            any_bad |= m.bad | (d & ~(u32)m.lead & 0xFFFFu & (m.oth | m.mark | m.spc | m.num | m.low | m.upp | m.cless));
        }
        if (tid < 2) {
            const long long chunk = tid == 0 ? c_first - 1 : c_first + TT_TILE_CHUNKS;
            ChunkMasks m = tt_classify_chunk(P.base, chunk, P.nchunks, P.lo, P.hi, T);
            const int s = tid == 0 ? 0 : TT_SLOTS - 1;
            sm[F_LEAD][s] = m.lead; sm[F_OTH][s] = m.oth; sm[F_MARK][s] = m.mark; sm[F_SPC][s] = m.spc;
            sm[F_NUM][s] = m.num; sm[F_LOW][s] = m.low; sm[F_UPP][s] = m.upp; sm[F_CLESS][s] = m.cless;
            sm[F_NL][s] = m.nl; sm[F_SP][s] = m.sp; sm[F_AP][s] = m.ap; sm[F_SL][s] = m.sl; sm[F_DOC][s] = (u16)doc_bits(P, chunk);
        }
        __syncthreads();
        // phase B: evaluate the piece-start predicate
        TileCarry tc; tc.n_before = 0; tc.nl_absorbed_before = 0; tc.nl_later_after = 0;
        u32 need = 0;
        const long long g0 = (c_first + tid) * TT_CHUNK;
        u32 S = P.pattern == 0 ? tt_eval_chunk_p0(sm, tid + 1, P.base, g0, P.hi, tc, false, need)
                               : tt_eval_chunk_p1(sm, tid + 1, P.base, g0, P.hi, tc, false, need);
        if (need) atomicOr(&s_need, need);
        __syncthreads();
        const u32 need_all = s_need;
        if (need_all) {                                               // block-uniform
            u32 a = 0, b = 0, c = 0;
            if (need_all & NEED_N) a = coop_back_num(P, T, c_first - 1, scratch);
            if (need_all & NEED_A) b = coop_back_nl(P, T, c_first - 1, scratch);
            if (need_all & NEED_F) c = coop_fwd_nl(P, T, c_first + TT_TILE_CHUNKS + 1, scratch);
            tc.n_before = a; tc.nl_absorbed_before = b; tc.nl_later_after = c;
            need = 0;
            S = P.pattern == 0 ? tt_eval_chunk_p0(sm, tid + 1, P.base, g0, P.hi, tc, true, need)
                               : tt_eval_chunk_p1(sm, tid + 1, P.base, g0, P.hi, tc, true, need);
        }
        if (c_first + tid < P.nchunks) P.startmask[c_first + tid] = (u16)S;
        u32 total = cta_sum_u32(tt_popc(S), scratch);
        if (tid == 0) P.tile_cnt[tile] = total;
    }
    if (any_bad) atomicMax(&P.hdr->status, 4 /* TT_ERR_INVALID_UTF8 */);

    // the last CTA to finish turns the tile counts into their exclusive prefix
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

// ---- K3: compaction of the start flags into piece offsets ---------------------------------------
// piece_off[i] = byte offset (relative to the text) of piece i; piece_off[n_pieces] = len.
__global__ void __launch_bounds__(TT_TILE_CHUNKS)
k_compact(const u16* __restrict__ startmask, const u32* __restrict__ tile_base, long long nchunks, int ntiles,
          long long shift, long long len, u32* __restrict__ piece_off, TTHeader* hdr) {
    __shared__ u32 sc[40];
    if (hdr->status != 0) return;
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

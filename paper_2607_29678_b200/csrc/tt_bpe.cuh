// Steps K4 and K5: byte-level BPE per piece, token counts and scatter of the IDs.
//
// Paper Sec. 4.2: every piece is encoded independently; merge ranks and vocabulary entries live in
// GPU hash tables; a round's minimum rank identifies one pair value, merging all its leftmost
// non-overlapping occurrences equals iterated single merges, and only pairs next to a completed
// merge need to be probed again.  Work is dispatched by piece length and difficulty:
//   * the first kernel (k_pretok, fused) has looked every piece up as a whole vocabulary entry (one 32-byte probe) and
//     left the others in its tile's queue region by length class;
//   * k_merge (a request) / k_closing + k_merge_bulk (bulk text): a warp per piece (<= 32 bytes: tokens in registers,
//     candidates as ballot masks; <= 256 bytes: several tokens per lane, compaction through shared memory), or, where
//     the call has many pieces of <= 32 bytes, 32 of them at once, a thread per piece (lane_merge); longer pieces
//     are merged by a whole CTA of 768 threads (cta_merge_long: state in shared memory, or in global scratch while
//     the piece still has more than 14,336 tokens).
// Token ids inside the kernels are "internal": byte b -> b, result of the merge of rank r -> 256 + r;
// the caller's ids are looked up when the tokens are staged.
//
// Rounds merge more than the minimum rank.  The sequential algorithm (always the leftmost pair of the lowest
// rank) performs a fixed set of merges on a piece; a round may perform any of them early, because the set, not
// the order, fixes the result.  A pair (t[i], t[i+1]) of rank r is certain to be in that set when neither token
// can be taken by another merge before rank r comes up:
//   * t[i] can only be taken from the left by a merge (X, t[i]) whose left operand X ends with the present
//     token t[i-1] (X is t[i-1] itself or was built on top of it).  cl(u, t) is the lowest rank of any
//     vocabulary merge (X, t) with u on the right spine of X's merge tree; the left guard is r < cl(t[i-1], t[i]);
//   * t[i+1] can only be taken from the right by a merge (t[i+1], Y) whose right operand begins with t[i+2].
//     cr(t, w) is the lowest rank of any merge (t, Y) with w on the left spine of Y; the right guard is
//     r <= cr(t[i+1], t[i+2]) (at equal rank the pair on the left comes first).
// Both guards are static properties of the vocabulary and are stored with the pair's rank, so one probe
// returns (rank, cl, cr) for a pair of adjacent tokens.  The pairs of the round's minimum rank need no guard
// (nothing can come before them).  In a run of identical pairs (t t t t ...) every other pair from a selected
// first one is selected, as in the sequential left-to-right order.  Everything selected in a round is merged
// at once; the result is the sequential one.
#pragma once
#include "tt_common.cuh"

// ---- pair table: (left, right) -> (rank, cl, cr) ----------------------------------------------------------
// Two-choice (cuckoo) hashing over buckets of two 16-byte slots (one 32-byte sector): a key is in one of its
// two buckets or nowhere, so a probe is two independent sector loads and no chain to walk, hit or miss.
// slot = { (left << 38) | (right << 20) | rank20, cl, cr } with rank20 = 0xFFFFF for a pair that is no merge
// itself (it is in the table for its guards); a free slot is all ones.
struct PairInfo { u32 r, cl, cr; };                   // TT_RANK_INF where there is none
struct PairTable {
    const uint4* slots;   // 2 * (mask + 1) slots
    const u64* bytepair;  // (byte a, byte b) at [a << 8 | b]: rank20 | cl20 << 20 | cr20 << 40 (0xFFFFF = none): a piece's first probes
    u32 mask;             // number of buckets - 1 (power of two, >= 256)
    u32 shift;            // 32 - log2(number of buckets)
};
constexpr u32 TT_F20 = 0xFFFFFu;                      // 20-bit field: none
TT_HD u32 f20_decode(u32 f) { return f == TT_F20 ? TT_RANK_INF : f; }
TT_HD u32 f20_encode(u32 r) { return r < TT_F20 ? r : TT_F20; }
TT_HD u32 pair_bucket(u64 key, u32 shift) {
    const u32 x = ((u32)key ^ ((u32)(key >> 32) * 0x9E3779B1u)) * 0x85EBCA6Bu;
    return (x ^ (x >> 15)) * 0xC2B2AE35u >> shift;
}
TT_HD u32 pair_bucket_alt(u64 key, u32 shift, u32 first) {      // the key's other bucket, never the first one
    u32 x = ((u32)(key >> TT_ID_BITS) * 0xCC9E2D51u) ^ ((u32)key * 0x1B873593u);
    x ^= x >> 16; x *= 0x7FEB352Du; x ^= x >> 15;
    const u32 h = (x * 0x846CA68Bu) >> shift;
    return h == first ? (first ^ 1u) : h;
}

__device__ __forceinline__ PairInfo pair_none() { PairInfo p; p.r = p.cl = p.cr = TT_RANK_INF; return p; }
__device__ __forceinline__ bool pair_match(const uint4 s, u64 key, PairInfo& out) {
    const u64 kr = ((u64)s.y << 32) | s.x;
    if ((kr >> 20) != key) return false;
    out.r = f20_decode((u32)kr & TT_F20); out.cl = s.z; out.cr = s.w;
    return true;
}

__device__ __forceinline__ PairInfo pair_probe(const PairTable& t, u32 a, u32 b) {
    const u64 key = ((u64)a << TT_ID_BITS) | b;
    const u32 h0 = pair_bucket(key, t.shift), h1 = pair_bucket_alt(key, t.shift, h0);
    const uint4* b0 = t.slots + 2 * (size_t)h0;
    const uint4* b1 = t.slots + 2 * (size_t)h1;
    const uint4 x0 = __ldg(b0), y0 = __ldg(b0 + 1), x1 = __ldg(b1), y1 = __ldg(b1 + 1);
    PairInfo out = pair_none();
    if (!pair_match(x0, key, out) && !pair_match(y0, key, out) && !pair_match(x1, key, out)) pair_match(y1, key, out);
    return out;
}
__device__ __forceinline__ PairInfo bytepair_info(const PairTable& t, u32 a, u32 b) {
    const u64 x = __ldg(t.bytepair + ((a << 8) | b));
    PairInfo p;
    p.r = f20_decode((u32)x & TT_F20); p.cl = f20_decode((u32)(x >> 20) & TT_F20); p.cr = f20_decode((u32)(x >> 40) & TT_F20);
    return p;
}

// Asks for [p, p + bytes) to be brought into L2, spread over the whole grid (no result, nothing waits for it).
// Used by a kernel while it waits for its predecessor: the tables it is about to probe at random are fetched
// with idle bandwidth, so that after a cold start its dependent loads find them in L2.
__device__ __forceinline__ void grid_prefetch_l2(const void* p, size_t bytes) {
    const char* c = reinterpret_cast<const char*>(p);
    const size_t lines = (bytes + 127) / 128, stride = (size_t)gridDim.x * blockDim.x;
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < lines; i += stride)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(c + i * 128));
}

// ---- whole-piece table: byte string of a vocabulary entry -> its id ------------------------------------
// Holds every token of at most TT_TOKTAB_MAXLEN bytes whose own byte string encodes to exactly that
// token (checked at load time by running the merge kernel below on every token string), so a hit
// returns what the merge loop would return.  Slots are 32 bytes (one sector): length (0 = empty), the
// caller's id and six key words (the bytes, little endian, zero padded); open addressing, linear probing,
// load factor <= 0.5.  The first 16 bytes of a slot (length, id, key words 0 and 1) decide every piece of at
// most 8 bytes -- most pieces of ordinary text -- with one vector load.
constexpr int TT_TOKTAB_MAXLEN = 24;
struct TokSlot { u32 len; int32_t id; u32 k[6]; };
static_assert(sizeof(TokSlot) == 32, "slot layout");
struct TokTable { const TokSlot* slots; u32 mask; u32 shift; };   // shift = 32 - log2(capacity)

// Key words beyond the piece are zero, so they add nothing: a piece of at most 8 bytes is hashed from two words.
TT_HD u32 toktab_hash_short(u32 k0, u32 k1, u32 n) { return n * 0x9E3779B1u + k0 * 0x85EBCA6Bu + k1 * 0xC2B2AE35u; }
TT_HD u32 toktab_hash_rest(u32 h, u32 k2, u32 k3, u32 k4, u32 k5) { return h + k2 * 0x27D4EB2Fu + k3 * 0x165667B1u + k4 * 0xD3A2646Du + k5 * 0xFD7046C5u; }
TT_HD u32 toktab_hash_final(u32 h, u32 shift) {
    h ^= h >> 15; h *= 0x2C1B3C6Du; h ^= h >> 12; h *= 0x297A2D39u; h ^= h >> 15;
    return h >> shift;
}
TT_HD u32 toktab_mask_word(u32 w, u32 n, u32 j) {      // key word j of a piece of n bytes: bytes beyond the piece are zero
    const u32 have = n > 4 * j ? n - 4 * j : 0u;
    return have >= 4 ? w : have == 0 ? 0u : w & ((1u << (8 * have)) - 1u);
}

#if defined(__CUDACC__)
// Key words 0 and 1 of the piece of n >= 1 bytes at text + a, from the aligned words x0, x1, x2 that hold it
// (x1 / x2 only where the piece reaches them).
__device__ __forceinline__ void toktab_key01(u32 x0, u32 x1, u32 x2, u32 sb, u32 n, u32& k0, u32& k1) {
    const u32 sh = sb * 8;
    k0 = toktab_mask_word(__funnelshift_r(x0, x1, sh), n, 0);
    k1 = toktab_mask_word(__funnelshift_r(x1, x2, sh), n, 1);
}
// Looks a piece of 2..24 bytes up; returns true and the id on a hit.  (The first kernel has its own copy of the
// first steps for pieces of at most 8 bytes, four pieces in flight per thread.)
__device__ __forceinline__ bool toktab_lookup(const TokTable& tab, const u8* __restrict__ text, u32 a, u32 n, int32_t& id) {
    const uintptr_t addr = (uintptr_t)(text + a);
    const u32* w = reinterpret_cast<const u32*>(addr & ~(uintptr_t)3);
    const u32 sb = (u32)(addr & 3), sh = sb * 8, used = sb + n;           // bytes of the aligned window that hold the piece
    u32 x[7];
#pragma unroll
    for (int j = 0; j < 7; j++) x[j] = used > 4u * j ? w[j] : 0u;          // only words that hold a piece byte (plain loads: the first kernel may have written the text itself)
    u32 k[6];
#pragma unroll
    for (int j = 0; j < 6; j++) k[j] = toktab_mask_word(__funnelshift_r(x[j], x[j + 1], sh), n, j);
    u32 h = toktab_hash_final(toktab_hash_rest(toktab_hash_short(k[0], k[1], n), k[2], k[3], k[4], k[5]), tab.shift);
    for (u32 probe = 0; probe <= tab.mask; probe++) {           // bounded by the capacity
        const uint4* sp = reinterpret_cast<const uint4*>(tab.slots + h);
        const uint4 lo = __ldg(sp);
        if (lo.x == 0) return false;
        if (lo.x == n && lo.z == k[0] && lo.w == k[1]) {
            bool same = true;
            if (n > 8) { const uint4 hi = __ldg(sp + 1); same = hi.x == k[2] && hi.y == k[3] && hi.z == k[4] && hi.w == k[5]; }
            if (same) { id = (int32_t)lo.y; return true; }
        }
        h = (h + 1) & tab.mask;
    }
    return false;
}
#endif

// ---- long-entry table (ignore_merges only): vocabulary entries of more than TT_TOKTAB_MAXLEN bytes --------
// Slot = (64-bit hash of the bytes, offset into a byte blob, length, id); open addressing, load <= 0.5.  A hit
// needs equal hash, equal length and equal bytes.
struct LongSlot { u64 hash; u32 off; u32 len; int32_t id; u32 pad; };
static_assert(sizeof(LongSlot) == 24, "slot layout");
struct LongTable { const LongSlot* slots; const u8* blob; u32 mask; u32 maxlen; };   // slots == nullptr: none

TT_HD u64 longtab_hash(const u8* p, u32 n) {
    u64 h = 0xCBF29CE484222325ull ^ n;
    for (u32 i = 0; i < n; i++) { h ^= p[i]; h *= 0x100000001B3ull; }
    h ^= h >> 32;
    return h * 0x9E3779B97F4A7C15ull;
}
__device__ __forceinline__ bool longtab_lookup(const LongTable& tab, const u8* __restrict__ text, u32 a, u32 n, int32_t& id) {
    const u64 h = longtab_hash(text + a, n);
    u32 s = (u32)(h >> 32) & tab.mask;
    for (u32 probe = 0; probe <= tab.mask; probe++) {             // bounded by the capacity
        const LongSlot e = tab.slots[s];
        if (e.len == 0) return false;
        if (e.hash == h && e.len == n) {
            u32 k = 0;
            while (k < n && tab.blob[e.off + k] == text[a + k]) k++;
            if (k == n) { id = e.id; return true; }
        }
        s = (s + 1) & tab.mask;
    }
    return false;
}

constexpr u32 RK_STALE = 0xFFFFFFFEu;                 // rank must be probed again
constexpr int BPE_WARPS = 8;                          // warps per CTA of the piece kernels
constexpr int BPE_THREADS = BPE_WARPS * 32;           // = pieces per CTA iteration
constexpr int WCH = TT_WARP_PIECE_MAX / 32;           // 32-token chunks per piece

// Position of the (j + 1)-th set bit of mask (a value >= 32 where there is none): five halving steps.
__device__ __forceinline__ u32 select_bit(u32 mask, u32 j) {
    u32 pos = 0, c;
    c = __popc(mask & 0xFFFFu);          if (j >= c) { pos = 16; j -= c; }
    c = __popc((mask >> pos) & 0xFFu);   if (j >= c) { pos += 8; j -= c; }
    c = __popc((mask >> pos) & 0xFu);    if (j >= c) { pos += 4; j -= c; }
    c = __popc((mask >> pos) & 0x3u);    if (j >= c) { pos += 2; j -= c; }
    c = (mask >> pos) & 1u;              if (j >= c) { pos += 1; j -= c; }
    return ((mask >> (pos & 31)) & 1u) && j == 0 && pos < 32 ? pos : 32u;
}

// ---- warp merge rounds with at most 32 tokens: one token per lane, no shared memory -----------------------
// t = token of position `lane`, p = (rank, cl, cr) of the pair (lane, lane + 1) or none, m = token count.
// Runs rounds to the fixpoint, stages the tokens (caller's ids) at stage[a ...] and returns their count.
// A round: Q marks a pair identical to the pair on its left (t t t); a pair that is not Q heads a run; a head
// may go if its left guard holds or it has the round's minimum rank; a pair goes if its run's head may go, it
// lies an even number of places behind the head and its right guard holds (or it has the minimum rank).
__device__ __forceinline__ u32 warp_merge_reg_rounds(u32 t, PairInfo p, u32 m, u32 a, const PairTable& tab,
                                                     const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage, int lane) {
    const u32 FULL = 0xFFFFFFFFu, lt = (1u << lane) - 1, le = lt | (1u << lane);
    u32 r = p.r, cl = p.cl, cr = p.cr;
    if ((u32)lane + 1 >= m) r = cl = cr = TT_RANK_INF;      // the last token has no pair
    const u32 max_rounds = m;                           // every round merges at least one pair
    for (u32 round = 0; round < max_rounds; round++) {
        const u32 mn = __reduce_min_sync(FULL, r);
        if (mn == TT_RANK_INF) break;
        const u32 tl = __shfl_up_sync(FULL, t, 1), tn0 = __shfl_down_sync(FULL, t, 1);
        u32 cll = __shfl_up_sync(FULL, cl, 1), crr = __shfl_down_sync(FULL, cr, 1);
        if (lane == 0) cll = TT_RANK_INF;
        if (lane == 31) crr = TT_RANK_INF;
        const bool R = r != TT_RANK_INF, Mn = r == mn;
        const bool Q = R && lane >= 1 && tl == t && t == tn0;
        const u32 qm = __ballot_sync(FULL, Q), hm = __ballot_sync(FULL, !Q && R && (r < cll || Mn));
        const u32 h = 31u - (u32)__clz(~qm & le);       // bit 0 of qm is never set
        const u32 sel = __ballot_sync(FULL, R && ((hm >> h) & 1) && !(((u32)lane - h) & 1) && (r <= crr || Mn));
        const bool me = (sel >> lane) & 1;
        const bool nxt = lane < 31 ? ((sel >> (lane + 1)) & 1) : false;
        const u32 nt = me ? 256u + r : t;
        const u32 nr = (me || nxt) ? RK_STALE : r;
        // survivors move down: new lane j takes the j-th surviving old lane
        u32 src;
        if ((sel & (sel - 1)) == 0) {                   // one merge: everything above it moves down by one
            src = (u32)lane + ((u32)lane > (u32)(__ffs(sel) - 1) ? 1u : 0u);
        } else {
            const u32 surv = ~(sel << 1) & (m >= 32 ? FULL : ((1u << m) - 1));
            src = select_bit(surv, (u32)lane);
        }
        t = __shfl_sync(FULL, nt, src & 31);
        r = __shfl_sync(FULL, nr, src & 31);
        cl = __shfl_sync(FULL, cl, src & 31);
        cr = __shfl_sync(FULL, cr, src & 31);
        m -= __popc(sel);
        const u32 tn = __shfl_down_sync(FULL, t, 1);
        if ((u32)lane + 1 >= m) r = cl = cr = TT_RANK_INF;
        else if (r == RK_STALE) { const PairInfo q = pair_probe(tab, t, tn); r = q.r; cl = q.cl; cr = q.cr; }
    }
    if ((u32)lane < m) stage[a + lane] = ext_id[t];
    return m;
}

// A piece of up to 32 bytes.
__device__ __forceinline__ u32 warp_merge_reg(const u8* __restrict__ text, u32 a, u32 n, const PairTable& tab,
                                              const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage, int lane) {
    const u32 t = (u32)lane < n ? text[a + lane] : 0;
    const u32 tn = __shfl_down_sync(0xFFFFFFFFu, t, 1);
    const PairInfo p = ((u32)lane + 1 < n) ? bytepair_info(tab, t, tn) : pair_none();
    return warp_merge_reg_rounds(t, p, n, a, tab, ext_id, stage, lane);
}

// ---- warp merge, 33..32 E bytes: E tokens per lane, compaction through shared memory ------------------------
// Position k lives in lane k % 32, register k / 32.  Shared memory holds two copies of four arrays of 32 E
// words (token, rank, cl, cr by position).  Each round the survivors are written to their new positions in
// the other copy and read back (one warp barrier); ranks next to a merge are marked stale and probed again,
// the probed guards go to the current copy, from which the next round reads its neighbours' values.
template <int E>
__device__ __forceinline__ u32 warp_merge_perm(u32* buf /* 2 * 4 * 32 E words of this warp */, const u8* __restrict__ text,
                                               u32 a, u32 n, const PairTable& tab, const int32_t* __restrict__ ext_id,
                                               int32_t* __restrict__ stage, int lane) {
    constexpr u32 N = 32 * E;
    const u32 FULL = 0xFFFFFFFFu, lt = (1u << lane) - 1, le = lt | (1u << lane);
    u32 t[E], r[E];
    u32 m = n;
    u32* cb = buf;                                      // current copy: tokens [0, N), ranks [N, 2N), cl [2N, 3N), cr [3N, 4N)
    u32* ob = buf + 4 * N;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < E; j++) {
        const u32 k = j * 32 + lane;
        t[j] = k < n ? text[a + k] : 0;
        cb[k] = t[j];
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < E; j++) {
        const u32 k = j * 32 + lane;
        const PairInfo p = (k + 1 < n) ? bytepair_info(tab, t[j], cb[k + 1]) : pair_none();
        r[j] = p.r; cb[2 * N + k] = p.cl; cb[3 * N + k] = p.cr;
    }
    for (u32 round = 0; round < n; round++) {          // at most n - 1 merges, at least one per round
        u32 mn = r[0];
#pragma unroll
        for (int j = 1; j < E; j++) mn = min(mn, r[j]);
        mn = __reduce_min_sync(FULL, mn);
        if (mn == TT_RANK_INF) break;
        __syncwarp();                                   // the guards written after the probes are visible
        if (m <= 32) {                                  // cheaper rounds from here on
            PairInfo p; p.r = r[0]; p.cl = cb[2 * N + lane]; p.cr = cb[3 * N + lane];
            return warp_merge_reg_rounds(t[0], p, m, a, tab, ext_id, stage, lane);
        }
        const int nch = (int)((m + 31) >> 5);
        u32 sel[E];
        u32 carry_hok = 0, carry_par = 0;               // head of the run that reaches into the word: may it go / parity of its position
#pragma unroll
        for (int j = 0; j < E; j++) {
            sel[j] = 0;
            if (j < nch) {
                const u32 k = j * 32 + lane;
                const bool R = r[j] != TT_RANK_INF, Mn = r[j] == mn;          // R implies k + 1 < m
                const u32 tl = k ? cb[k - 1] : 0xFFFFFFFFu, tn = R ? cb[k + 1] : 0xFFFFFFFEu;
                const u32 cll = k ? cb[2 * N + k - 1] : TT_RANK_INF;
                const u32 crr = (k + 2 < m) ? cb[3 * N + k + 1] : TT_RANK_INF;
                const bool Q = R && tl == t[j] && t[j] == tn;
                const u32 qm = __ballot_sync(FULL, Q), hm = __ballot_sync(FULL, !Q && R && (r[j] < cll || Mn));
                const u32 z = ~qm & le;
                u32 hok, par;
                if (z) { const u32 ph = 31u - (u32)__clz(z); hok = (hm >> ph) & 1; par = ((u32)lane - ph) & 1; }
                else { hok = carry_hok; par = ((u32)lane & 1) ^ carry_par; }
                sel[j] = __ballot_sync(FULL, R && hok && !par && (r[j] <= crr || Mn));
                if (~qm) { const u32 ph = 31u - (u32)__clz(~qm); carry_par = ph & 1; carry_hok = (hm >> ph) & 1; }
            }
        }
        u32 removed = 0;
#pragma unroll
        for (int j = 0; j < E; j++) {
            if (j < nch) {
                const u32 k = j * 32 + lane;
                const u32 s = sel[j];
                const bool me = (s >> lane) & 1;
                const bool gone = lane ? ((s >> (lane - 1)) & 1) : (j ? (sel[j > 0 ? j - 1 : 0] >> 31) & 1 : 0);
                const bool next_sel = lane < 31 ? ((s >> (lane + 1)) & 1) : ((j + 1 < E) ? (sel[j + 1 < E ? j + 1 : j] & 1) : 0);
                if (k < m && !gone) {
                    const u32 np = k - removed - __popc(s & lt);
                    ob[np] = me ? 256u + r[j] : t[j];
                    ob[N + np] = (me || next_sel) ? RK_STALE : r[j];
                    ob[2 * N + np] = cb[2 * N + k];
                    ob[3 * N + np] = cb[3 * N + k];
                }
                removed += __popc(s);
            }
        }
        m -= removed;
        { u32* x = cb; cb = ob; ob = x; }
        __syncwarp();
#pragma unroll
        for (int j = 0; j < E; j++) {
            const u32 k = j * 32 + lane;
            r[j] = TT_RANK_INF;
            if (k < m) {
                t[j] = cb[k];
                r[j] = cb[N + k];
                if (k + 1 >= m) r[j] = TT_RANK_INF;
                else if (r[j] == RK_STALE) {
                    const PairInfo p = pair_probe(tab, t[j], cb[k + 1]);
                    r[j] = p.r; cb[2 * N + k] = p.cl; cb[3 * N + k] = p.cr;
                }
            }
        }
    }
#pragma unroll
    for (int j = 0; j < E; j++) {
        const u32 k = j * 32 + lane;
        if (k < m) stage[a + k] = ext_id[t[j]];
    }
    return m;
}

// ---- a thread per piece, <= 32 bytes: tokens and pair ranks in shared memory ------------------------------
// Paper Sec. 4.2 gives the shortest length class to single threads.  Here a warp per piece has the shorter
// dependent chain (one probe latency per round for the whole piece), so it serves a request's few
// unmatched pieces; a thread per piece keeps 32 independent chains per warp in flight and issues an order
// of magnitude fewer instructions per piece, so it serves bulk text.  Same rounds as everywhere: the
// minimum rank of the piece, all its leftmost non-overlapping occurrences, new probes only next to a merge.
// Column s of tok[LANE_MAX][LANE_SLOTS] / rk[LANE_MAX][LANE_SLOTS] (one pair of arrays per warp): any two
// threads of the warp hit different banks whatever rows they are at.
constexpr int LANE_SLOTS = 32;                        // pieces a warp merges at once
constexpr int LANE_MAX = 32;                          // bytes per piece on this path
// Two independent probes (ranks only), all loads in flight together.
__device__ __forceinline__ void pair_probe2(const PairTable& t, u32 a0, u32 b0, u32 a1, u32 b1, u32& r0, u32& r1) {
    const u64 key0 = ((u64)a0 << TT_ID_BITS) | b0, key1 = ((u64)a1 << TT_ID_BITS) | b1;
    const u32 h00 = pair_bucket(key0, t.shift), h01 = pair_bucket_alt(key0, t.shift, h00);
    const u32 h10 = pair_bucket(key1, t.shift), h11 = pair_bucket_alt(key1, t.shift, h10);
    const uint4* p00 = t.slots + 2 * (size_t)h00; const uint4* p01 = t.slots + 2 * (size_t)h01;
    const uint4* p10 = t.slots + 2 * (size_t)h10; const uint4* p11 = t.slots + 2 * (size_t)h11;
    const uint4 a00 = __ldg(p00), a01 = __ldg(p00 + 1), a02 = __ldg(p01), a03 = __ldg(p01 + 1);
    const uint4 a10 = __ldg(p10), a11 = __ldg(p10 + 1), a12 = __ldg(p11), a13 = __ldg(p11 + 1);
    PairInfo q0 = pair_none(), q1 = pair_none();
    if (!pair_match(a00, key0, q0) && !pair_match(a01, key0, q0) && !pair_match(a02, key0, q0)) pair_match(a03, key0, q0);
    if (!pair_match(a10, key1, q1) && !pair_match(a11, key1, q1) && !pair_match(a12, key1, q1)) pair_match(a13, key1, q1);
    r0 = q0.r; r1 = q1.r;
}

// Tokens stay at the byte position where they began; `al` has a bit per position that still holds a
// token, and the rank of a pair is kept at its left position, so a merge moves nothing: it rewrites the
// left token, clears the partner's bit and marks the two pairs that changed for a new probe.
__device__ __forceinline__ u32 lane_merge(u32* __restrict__ tok, u32* __restrict__ rk, int s, const u8* __restrict__ text, u32 a, u32 n,
                                          const PairTable& tab, const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage) {
#define TK(k) tok[(k) * LANE_SLOTS + s]
#define RK(k) rk[(k) * LANE_SLOTS + s]
    u32 prev = text[a];
    TK(0) = prev;
#pragma unroll 4
    for (u32 k = 1; k < n; k++) {
        const u32 t = text[a + k];
        TK(k) = t;
        RK(k - 1) = f20_decode((u32)__ldg(tab.bytepair + ((prev << 8) | t)) & TT_F20);
        prev = t;
    }
    u32 al = 0xFFFFFFFFu >> (32 - n);
    u32 stale = 0;
    for (u32 round = 0; round < n; round++) {
        while (stale) {                                   // every thread of the warp walks its own list in step
            const u32 k0 = __ffs(stale) - 1;
            stale &= stale - 1;
            const u32 k1 = stale ? __ffs(stale) - 1 : k0;
            stale &= stale - 1;
            const u32 up0 = al & (0xFFFFFFFEu << k0), up1 = al & (0xFFFFFFFEu << k1);
            u32 r0 = TT_RANK_INF, r1 = TT_RANK_INF;         // (a position without a token above it has no pair)
            pair_probe2(tab, TK(k0), up0 ? TK(__ffs(up0) - 1) : 0u, TK(k1), up1 ? TK(__ffs(up1) - 1) : 0u, r0, r1);
            RK(k0) = up0 ? r0 : TT_RANK_INF;
            RK(k1) = up1 ? r1 : TT_RANK_INF;
        }
        u32 mn = TT_RANK_INF, c = 0;
        for (u32 x = al & ~(0x80000000u >> __clz(al)); x; x &= x - 1) {      // every position but the topmost
            const u32 k = __ffs(x) - 1;
            const u32 r = RK(k);
            if (r < mn) { mn = r; c = 0; }
            c |= (r == mn ? 1u : 0u) << k;
        }
        if (mn == TT_RANK_INF) break;
        const u32 nt = 256u + mn;
        u32 blocked = 32;
        for (u32 x = c; x; x &= x - 1) {                  // leftmost non-overlapping occurrences, ascending
            const u32 k = __ffs(x) - 1;
            if (k == blocked) continue;                   // its token went into the merge before it
            const u32 p = __ffs(al & (0xFFFFFFFEu << k)) - 1;
            TK(k) = nt;
            al &= ~(1u << p);
            blocked = p;
            const u32 below = al & ((1u << k) - 1);
            stale |= (1u << k) | (below ? 0x80000000u >> __clz(below) : 0u);
        }
    }
    u32 m = 0;
    for (u32 x = al; x; x &= x - 1) stage[a + m++] = ext_id[TK(__ffs(x) - 1)];
#undef TK
#undef RK
    return m;
}

// ---- CTA-wide helpers ------------------------------------------------------------------------------------
__device__ __forceinline__ u32 cta_excl_sum_scan(u32 v, u32* scratch /* >= 33 */, u32* total) {
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
    *total = scratch[32];
    return scratch[wid] + x - v;
}
// Sums of two values over the CTA, returned to every thread (scratch >= 66 entries; two barriers).
__device__ __forceinline__ void cta_sum2_u64(unsigned long long& x, unsigned long long& y, unsigned long long* scratch) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
    for (int o = 16; o; o >>= 1) { x += __shfl_xor_sync(0xFFFFFFFFu, x, o); y += __shfl_xor_sync(0xFFFFFFFFu, y, o); }
    __syncthreads();
    if (lane == 0) { scratch[2 * wid] = x; scratch[2 * wid + 1] = y; }
    __syncthreads();
    x = 0; y = 0;
    for (int w = 0; w < nw; w++) { x += scratch[2 * w]; y += scratch[2 * w + 1]; }
}

__device__ __forceinline__ u32 cta_min_u32(u32 v, u32* scratch /* >= 33 */) {
    v = __reduce_min_sync(0xFFFFFFFFu, v);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
    __syncthreads();
    u32 r = scratch[0];
    for (int w = 1; w < (int)(blockDim.x >> 5); w++) r = min(r, scratch[w]);
    return r;
}

// ---- CTA merge for long pieces -----------------------------------------------------------------------------
// arr[i] = token | rank20 << 18 | cl20 << 38 and crr[i] = cr20 for position i (rank and guards of the pair
// (i, i + 1); 20-bit fields, 0xFFFFF = none), in global scratch or shared memory.  One round: the minimum rank
// is found, every thread takes LK consecutive positions and decides which of its pairs are merged (same rule
// as in the warp rounds; the state of a run of identical pairs that crosses slices -- may its head go, parity
// of the distance to it -- is carried from thread to thread with one ballot-based scan; LK is even, so a
// slice that lies inside one run passes the state on unchanged), and the survivors are written to their new
// positions in place, chunk after chunk (every thread of a chunk has its positions in registers before
// anything is written, and writes never pass the read front).  Ranks next to a merge are marked stale and
// probed again in a second sweep, which also yields the next round's minimum.
#ifndef TT_LK
#define TT_LK 6        // measured with 768 threads: 64 KB of random letters 94 ms at 16, 59 at 8, 45 at 6, 51 at 4, 59 at 2
#endif
constexpr int LK = TT_LK;                               // positions per thread and chunk (even)
// words of the CTA's scratch array: [0, 33) block scans and per-warp run states, then per-warp "last position merged" flags,
// the carried token / guard of a chunk's last position, and two words for broadcasts
constexpr int SCR_LASTM = 40, SCR_CARRY_TOK = 72, SCR_CARRY_CL = 73, SCR_FLAG = 74, SCR_VALUE = 75, SCR_WORDS = 80;
constexpr u32 F20_STALE = 0xFFFFEu;
TT_HD u64 lp_pack(u32 t, u32 r20, u32 cl20) { return (u64)t | ((u64)r20 << TT_ID_BITS) | ((u64)cl20 << (TT_ID_BITS + 20)); }
TT_HD u32 lp_tok(u64 v) { return (u32)v & (TT_MAX_INTERNAL - 1); }
TT_HD u32 lp_rank(u64 v) { return (u32)(v >> TT_ID_BITS) & TT_F20; }
TT_HD u32 lp_cl(u64 v) { return (u32)(v >> (TT_ID_BITS + 20)) & TT_F20; }

// padshift: 4 for arrays in shared memory (index i lives at i + i / 16: the slices of LK consecutive positions that the
// threads of a warp read then spread over more banks), 31 for arrays in global scratch (no padding).
#define AX(i) ((i) + ((i) >> padshift))
__device__ __noinline__ u32 cta_merge_rounds(u64* arr, u32* crr, u32 m, const PairTable& tab, u32* s_scr /* SCR_WORDS */, u32 stop_at, bool& finished, u32 padshift,
                                           u64* stg_a = nullptr, u32* stg_c = nullptr) {
    const int tid = threadIdx.x, T = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = T >> 5;
    const u32 FULL = 0xFFFFFFFFu, inmask = (1u << LK) - 1;
    finished = false;
    // minimum rank of the current array
    u32 lmin = TT_F20;
    for (u32 i0 = tid; i0 < m; i0 += (u32)T * 8) {
        u64 xs[8];
#pragma unroll
        for (int u = 0; u < 8; u++) { const u32 i = i0 + (u32)u * T; xs[u] = i < m ? arr[AX(i)] : lp_pack(0, TT_F20, TT_F20); }
#pragma unroll
        for (int u = 0; u < 8; u++) lmin = min(lmin, lp_rank(xs[u]));
    }
    for (;;) {
        const u32 mn = cta_min_u32(lmin, s_scr);
        if (mn >= F20_STALE) { finished = true; return m; }
        if (m <= stop_at) return m;
        u32 carry_hok = 0, carry_par = 0, carry_last = 0, out = 0;    // run state and last selection before the chunk; survivors so far
        for (u32 base = 0; base < m; base += (u32)T * LK) {
            const u32 i0 = base + (u32)tid * LK;
            u64 v[LK + 3];                                  // positions i0 - 1 .. i0 + LK + 1
            u32 c[LK + 3];
#pragma unroll
            for (int k = 0; k < LK + 3; k++) {
                const u32 i = i0 + k - 1;                   // wraps for position -1 of the piece: not below m
                v[k] = lp_pack(0, TT_F20, TT_F20); c[k] = TT_F20;
                if (k == 0 && tid == 0) { if (base) v[k] = lp_pack(s_scr[SCR_CARRY_TOK], TT_F20, s_scr[SCR_CARRY_CL]); }   // overwritten by the chunk before: carried
                else if (i < m) { v[k] = arr[AX(i)]; c[k] = crr[AX(i)]; }
            }
            const u32 nval = i0 < m ? min((u32)LK, m - i0) : 0;
            u32 Qm = 0, Hm = 0, Gm = 0;                     // bit k: position i0 + k, k = 0 .. LK
#pragma unroll
            for (int k = 0; k <= LK; k++) {
                const u32 rr = lp_rank(v[k + 1]), tk = lp_tok(v[k + 1]);
                const bool R = rr < F20_STALE, Mn = rr == mn;
                const bool Q = R && (i0 + k >= 1) && lp_tok(v[k]) == tk && tk == lp_tok(v[k + 2]);
                Qm |= (u32)Q << k;
                Hm |= (u32)(!Q && R && (rr < lp_cl(v[k]) || Mn)) << k;
                Gm |= (u32)(R && (rr <= c[k + 2] || Mn)) << k;
            }
            // state handed to the next slice: from my highest pair that heads a run
            const u32 nq = ~Qm & inmask;
            const bool all = nq == 0;
            u32 out_hok = 0, out_par = 0;
            if (nq) { const u32 ph = 31u - (u32)__clz(nq); out_hok = (Hm >> ph) & 1; out_par = ((u32)LK - ph) & 1; }
            const u32 allm = __ballot_sync(FULL, all), hokm = __ballot_sync(FULL, out_hok), parm = __ballot_sync(FULL, out_par);
            const u32 lower = ~allm & ((1u << lane) - 1);
            __syncthreads();
            if (lane == 31) {
                const u32 na = ~allm;
                u32 e = 0;
                if (na) { const u32 src = 31u - (u32)__clz(na); e = 4u | (((hokm >> src) & 1) << 1) | ((parm >> src) & 1); }
                s_scr[wid] = e;                              // 0 = all lanes pass through
            }
            __syncthreads();
            u32 in_hok, in_par;
            if (lower) { const u32 src = 31u - (u32)__clz(lower); in_hok = (hokm >> src) & 1; in_par = (parm >> src) & 1; }
            else {
                in_hok = carry_hok; in_par = carry_par;
                for (int w = wid - 1; w >= 0; w--) { const u32 e = s_scr[w]; if (e) { in_hok = (e >> 1) & 1; in_par = e & 1; break; } }
            }
            u32 next_hok = carry_hok, next_par = carry_par;
            for (int w = nw - 1; w >= 0; w--) { const u32 e = s_scr[w]; if (e) { next_hok = (e >> 1) & 1; next_par = e & 1; break; } }
            // selection inside the slice (positions 0..LK; position LK only to know whether it is merged)
            u32 sel = 0;
            {
                u32 hok = in_hok, par = in_par;
#pragma unroll
                for (int k = 0; k <= LK; k++) {
                    if (!((Qm >> k) & 1)) { hok = (Hm >> k) & 1; par = 0; }
                    sel |= (((Gm >> k) & 1) & hok & (par ^ 1u)) << k;
                    par ^= 1u;
                }
            }
            // was the position before my slice merged with my first one?
            const u32 lastm = __ballot_sync(FULL, (sel >> (LK - 1)) & 1);
            if (lane == 31) s_scr[SCR_LASTM + wid] = lastm >> 31;
            if (tid == T - 1) { s_scr[SCR_CARRY_TOK] = lp_tok(v[LK]); s_scr[SCR_CARRY_CL] = lp_cl(v[LK]); }     // position i0 + LK - 1 as it is now
            __syncthreads();
            const u32 gone0 = lane ? (lastm >> (lane - 1)) & 1 : (wid ? s_scr[SCR_LASTM + wid - 1] : carry_last);
            const u32 next_last = s_scr[SCR_LASTM + nw - 1];
            const u32 gone = ((sel << 1) | gone0) & inmask;
            const u32 valid = nval >= LK ? inmask : ((1u << nval) - 1);
            const u32 surv = valid & ~gone;
            u32 tot;
            const u32 ex = cta_excl_sum_scan(__popc(surv), s_scr, &tot);         // all loads of the chunk are done: barrier inside
            // Arrays in global scratch: the chunk's survivors are collected in shared memory and written out with
            // coalesced stores (a thread storing its own run of positions touches a line per store and lane, which
            // is what a chunk spent most of its time on).
            u64* const wa = stg_a ? stg_a : arr;
            u32* const wc = stg_a ? stg_c : crr;
            u32 o = stg_a ? ex : out + ex;
#pragma unroll
            for (int k = 0; k < LK; k++) {
                if ((surv >> k) & 1) {
                    const bool me = (sel >> k) & 1;
                    const bool nxt = me ? false : ((sel >> (k + 1)) & 1);
                    const u64 x = v[k + 1];
                    const u32 oi = stg_a ? o : AX(o);
                    wa[oi] = lp_pack(me ? 256u + lp_rank(x) : lp_tok(x), (me || nxt) ? F20_STALE : lp_rank(x), lp_cl(x));
                    wc[oi] = c[k + 1];
                    o++;
                }
            }
            if (stg_a) {
                __syncthreads();
                for (u32 e = tid; e < tot; e += T) { arr[out + e] = stg_a[e]; crr[out + e] = stg_c[e]; }
            }
            out += tot;
            carry_hok = next_hok; carry_par = next_par; carry_last = next_last;
            __syncthreads();
        }
        m = out;
        __syncthreads();
        // probe the stale ranks again; collect the minimum for the next round
        // (eight loads in flight per thread: in global scratch every one of them is an L2 round trip)
        lmin = TT_F20;
        for (u32 i0 = tid; i0 < m; i0 += (u32)T * 8) {
            u64 xs[8];
#pragma unroll
            for (int u = 0; u < 8; u++) { const u32 i = i0 + (u32)u * T; xs[u] = i < m ? arr[AX(i)] : lp_pack(0, TT_F20, TT_F20); }
#pragma unroll
            for (int u = 0; u < 8; u++) {
                const u32 i = i0 + (u32)u * T;
                const u64 x = xs[u];
                u32 r = lp_rank(x);
                if (i < m) {
                    if (i + 1 >= m) { r = TT_F20; arr[AX(i)] = lp_pack(lp_tok(x), TT_F20, TT_F20); crr[AX(i)] = TT_F20; }
                    else if (r == F20_STALE) {
                        const PairInfo p = pair_probe(tab, lp_tok(x), lp_tok(arr[AX(i + 1)]));
                        r = f20_encode(p.r);
                        arr[AX(i)] = lp_pack(lp_tok(x), r, f20_encode(p.cl)); crr[AX(i)] = f20_encode(p.cr);
                    }
                }
                lmin = min(lmin, r);
            }
        }
        __syncthreads();
    }
}

#ifndef TT_LONG_SMEM_TOKENS
#define TT_LONG_SMEM_TOKENS 14336
#endif
constexpr int LONG_SMEM_TOKENS = TT_LONG_SMEM_TOKENS;   // long pieces move into shared memory below this many tokens
constexpr int LONG_SMEM_SLOTS = LONG_SMEM_TOKENS + LONG_SMEM_TOKENS / 16 + 8;   // with the padding of the shared-memory layout; also holds a chunk's survivors


// Encodes one piece of n > TT_WARP_PIECE_MAX bytes with the whole CTA.  gbuf: n entries of global scratch; the
// piece's own n words of the staging array serve as the second global array until the ids are staged there.
// sbuf: LONG_SMEM_SLOTS u64 followed by LONG_SMEM_SLOTS u32.
__device__ u32 cta_merge_long(const u8* __restrict__ text, u32 a, u32 n, const PairTable& tab, const int32_t* __restrict__ ext_id,
                              int32_t* __restrict__ stage, u64* gbuf, u64* sbuf, u32* s_scr) {
    const int tid = threadIdx.x, T = blockDim.x;
    u32* const scr = reinterpret_cast<u32*>(sbuf + LONG_SMEM_SLOTS);
    u32* const gcr = reinterpret_cast<u32*>(stage + a);
    u64* arr = n <= LONG_SMEM_TOKENS ? sbuf : gbuf;
    u32* crr = n <= LONG_SMEM_TOKENS ? scr : gcr;
    u32 padshift = n <= LONG_SMEM_TOKENS ? 4u : 31u;
    __syncthreads();
    for (u32 i = tid; i < n; i += T) {
        const u32 t0 = text[a + i];
        const PairInfo p = (i + 1 < n) ? bytepair_info(tab, t0, text[a + i + 1]) : pair_none();
        arr[AX(i)] = lp_pack(t0, f20_encode(p.r), f20_encode(p.cl));
        crr[AX(i)] = f20_encode(p.cr);
    }
    __syncthreads();
    bool finished;
    u32 m = cta_merge_rounds(arr, crr, n, tab, s_scr, arr == gbuf ? LONG_SMEM_TOKENS : 0, finished, padshift,
                             arr == gbuf ? sbuf : nullptr, arr == gbuf ? scr : nullptr);       // the shared buffer stages the stores meanwhile
    if (!finished && arr == gbuf) {
        __syncthreads();
        padshift = 4u;
        for (u32 i = tid; i < m; i += T) { sbuf[AX(i)] = gbuf[i]; scr[AX(i)] = gcr[i]; }
        __syncthreads();
        arr = sbuf;
        m = cta_merge_rounds(arr, scr, m, tab, s_scr, 0, finished, padshift);
    }
    __syncthreads();
    for (u32 i = tid; i < m; i += T) stage[a + i] = ext_id[lp_tok(arr[AX(i)])];
    __syncthreads();
    return m;
}
#undef AX

// ---- what the first kernel (tag + piece starts + whole-piece lookups) leaves per tile -----------------------
// See TTWorkspace.  A queue entry of a tile names one unsettled piece of at most 256 bytes that lies inside the
// tile: offset in the tile | index among the tile's pieces << 11 | (bytes - 1) << 22.  The tile's LAST piece is
// never settled by the first kernel (its end is the next piece start, which another CTA finds): k_merge
// settles it, looking the end up in tile_first of the following tiles.
__device__ __forceinline__ u32 tile_queue_entry(u32 off, u32 idx, u32 n) { return off | (idx << 11) | ((n - 1) << 22); }
constexpr u32 TQ_NS_MASK = 0x7FFu, TQ_NW_SHIFT = 11, TQ_NW_MASK = 0x7Fu, TQ_NL_SHIFT = 18, TQ_NL_MASK = 0xFu;

struct PieceParams {
    const u8* base;            // aligned frame origin (text = base + shift)
    long long shift, hi;       // text occupies [shift, hi)
    int ntiles;
    const u32* tile_cnt;
    const u32* tile_first;
    const u32* tile_last;
    const u32* tile_q;
    const u16* tile_long;
    const u16* piece_off16;
    const u32* q;
    TTHeader* hdr;
    unsigned long long epoch;
    PairTable tab;
    TokTable toktab;           // slots == nullptr: no whole-piece table (while the table itself is being built)
    const u32* litstart;       // literal pass: a piece that begins at such a bit is an added token whose id is staged, or null
    LongTable longtab;         // ignore_merges: entries longer than the whole-piece table holds (else slots == nullptr)
    const int32_t* ext_id;
    u32* piece_cnt;
    int32_t* stage;            // ids staged at the text offset of their piece
    u64* pairbuf;              // global scratch of the long-piece path, indexed like the text
    u32* tile_tok;
    u32* grp_tok;              // bulk text: tokens per group of TT_GROUP_TILES tiles (written by the last CTA), else null
    u64* wq;                   // bulk text: the warp-class pieces of all tiles (tile << 32 | queue entry), else null
    u64* gq;                   // bulk text: the short pieces of all tiles, gathered by k_closing (tile << 32 | queue entry),
    u64* gq_x[3];              // one list per length class (tt_short_class_max); gq is the first
    uint4* lq;                 // bulk text: the long pieces of all tiles, listed by k_closing (text offset, bytes, piece slot, 0)
};

// ---- K4, second half: the merges ------------------------------------------------------------------------------
// Work of this kernel: the unsettled pieces the first kernel queued per tile, and the last piece of every tile.
//   (A) pieces of more than 256 bytes, a whole CTA each: every CTA looks through a contiguous share of the
//       tiles (the in-tile long pieces the first kernel listed, and tile-closing pieces that turn out long).
//   (B) everything else, warp by warp, without any barrier:
//       - a request (few tiles, few unsettled pieces): job j belongs to warp j of the grid.  Jobs are numbered
//         warp-class pieces first (the longest chains), then the tile-closing pieces, then the short pieces;
//         a warp finds its job from the per-tile counts alone (every lane sums a stretch of tiles, one warp
//         scan), so nothing is handed out through a counter.  One warp per piece, tokens in registers.
//       - bulk text: the warp-class pieces stand in one global list (they come in clusters; a list lets every warp
//         take its share), then warps draw tickets of one tile and settle its short pieces 32 at a time, a thread
//         each (lane_merge); pieces wait in the lanes across tickets until 32 are together.
#ifndef TT_MERGE_WARPS
#define TT_MERGE_WARPS 24
#endif
constexpr int MERGE_WARPS = TT_MERGE_WARPS;           // one CTA per SM: a long piece gets all its 768 threads and 192 KiB
constexpr int MERGE_THREADS = MERGE_WARPS * 32;
constexpr int WARP_SMEM_WORDS = 1024;                 // u64 per warp: two lane-path arrays of 32 x 32 u32, or two copies of four 256-word merge arrays
static_assert(MERGE_WARPS * WARP_SMEM_WORDS * sizeof(u64) >= LONG_SMEM_SLOTS * (sizeof(u64) + sizeof(u32)), "the CTA's buffer must hold a long piece");
static_assert(LONG_SMEM_TOKENS >= MERGE_WARPS * 32 * LK, "the survivors of a chunk (threads x LK positions) must fit the shared buffer");
constexpr size_t MERGE_SMEM_BYTES = (size_t)MERGE_WARPS * WARP_SMEM_WORDS * sizeof(u64);   // dynamic shared memory of k_merge (64 KiB)
static_assert(WARP_SMEM_WORDS * sizeof(u64) >= 2 * LANE_SLOTS * LANE_MAX * sizeof(u32) && WARP_SMEM_WORDS * sizeof(u64) >= 2 * 4 * TT_WARP_PIECE_MAX * sizeof(u32), "per-warp buffer");
constexpr int MERGE_SR_MAX_TILES = 2048;              // the per-warp job search covers at most 32 lanes x 64 tiles

#ifndef TT_MERGE_CTAS_PER_SM
#define TT_MERGE_CTAS_PER_SM 1
#endif
constexpr int MERGE_CTAS_PER_SM = TT_MERGE_CTAS_PER_SM;   // resident CTAs per SM (registers and the 64 KiB of shared memory each)

// End (aligned frame) of the piece that starts last in `tile`: the first piece start of a later tile, or the text end.
__device__ __forceinline__ u32 closing_piece_end(const PieceParams& P, int tile) {
    for (int t = tile + 1; t < P.ntiles; t++) {                   // bounded by the number of tiles
        const u32 f = P.tile_first[t];
        if (f != TT_NONE) return (u32)t * TT_TILE_BYTES + f;
    }
    return (u32)P.hi;
}

// A piece that needs no merging: an extracted literal (its id is staged already), a single byte, or a whole
// vocabulary entry.  Returns true and the value for piece_cnt.  One thread.
__device__ __forceinline__ bool piece_settled_without_merge(const PieceParams& P, const u8* __restrict__ text, u32 a, u32 n, u32& value) {
    if (P.litstart != nullptr) {
        const long long g = (long long)a + P.shift;
        if ((P.litstart[g >> 5] >> (g & 31)) & 1) { value = 0u - 1u; return true; }
    }
    int32_t id;
    if (n == 1) { value = (u32)P.ext_id[text[a]]; return true; }
    if (n <= TT_TOKTAB_MAXLEN) {
        if (P.toktab.slots != nullptr && toktab_lookup(P.toktab, text, a, n, id)) { value = (u32)id; return true; }
    } else if (P.longtab.slots != nullptr && n <= P.longtab.maxlen && longtab_lookup(P.longtab, text, a, n, id)) { value = (u32)id; return true; }
    return false;
}

__device__ __forceinline__ void piece_done(const PieceParams& P, u32 slot, u32 m) {
    P.piece_cnt[slot] = 0u - m;
    atomicAdd(&P.tile_tok[slot / TT_TILE_BYTES], m);
}

// One piece of 2..256 bytes, the whole warp.
__device__ __forceinline__ bool piece_in_range(const PieceParams& P, u32 a, u32 n, u32 slot, u32 site) {
    const bool ok = n >= 1 && (long long)a + n <= P.hi - P.shift && slot < (u32)P.ntiles * TT_TILE_BYTES;
    if (!ok) hdr_selfcheck_failed(P.hdr, P.epoch, site, a, n, slot, 0u);
    return ok;
}
__device__ __forceinline__ void warp_merge_piece(const PieceParams& P, const u8* __restrict__ text, u32 a, u32 n, u32 slot, u64* wbuf, int lane) {
    if (!piece_in_range(P, a, n, slot, 1u) || n < 2 || n > (u32)TT_WARP_PIECE_MAX) { if (n < 2 || n > (u32)TT_WARP_PIECE_MAX) hdr_selfcheck_failed(P.hdr, P.epoch, 2u, a, n, slot, 0u); return; }
    u32* const pbuf = reinterpret_cast<u32*>(wbuf);
    const u32 m = n <= LANE_MAX ? warp_merge_reg(text, a, n, P.tab, P.ext_id, P.stage, lane)
                : n <= 64 ? warp_merge_perm<2>(pbuf, text, a, n, P.tab, P.ext_id, P.stage, lane)
                : n <= 128 ? warp_merge_perm<4>(pbuf, text, a, n, P.tab, P.ext_id, P.stage, lane)
                           : warp_merge_perm<WCH>(pbuf, text, a, n, P.tab, P.ext_id, P.stage, lane);
    if (lane == 0) piece_done(P, slot, m);
}

// Exclusive prefix over the lanes of a 64-bit value holding two counts (low 32 bits, high 32 bits); *total = warp sum.
__device__ __forceinline__ u64 warp_exscan_u64(u64 v, int lane, u64* total) {
    u64 x = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const u64 t = __shfl_up_sync(0xFFFFFFFFu, x, o); if (lane >= o) x += t; }
    *total = __shfl_sync(0xFFFFFFFFu, x, 31);
    return x - v;
}

// ---- bulk text only: the closing pieces, and one list per length class for the whole text ---------------------
// A thread per tile settles the tile's closing piece where no merging is needed and gathers what is left of the
// 32 tiles of its warp -- queued short pieces, a short closing piece -- into one global list (one reservation
// per warp), so that k_merge's warps take 32 short pieces at a time whatever tile they come from; warp-class
// closing pieces join the first kernel's list, long pieces get a list of their own.  The counters were cleared
// by the memset in front of the chain.
constexpr int CLOSING_THREADS = 256;
// Length class of a short piece (2..32 bytes).
__device__ __forceinline__ int short_class(u32 n) {
    return n <= (u32)tt_short_class_max(0) ? 0 : n <= (u32)tt_short_class_max(1) ? 1 : n <= (u32)tt_short_class_max(2) ? 2 : 3;
}

__global__ void __launch_bounds__(CLOSING_THREADS)
k_closing(const PieceParams P) {
    const int lane = threadIdx.x & 31;
    const u32 FULL = 0xFFFFFFFFu;
    cudaTriggerProgrammaticLaunchCompletion();
    cudaGridDependencySynchronize();                         // the first kernel's per-tile records are complete from here on
    if (hdr_status(P.hdr, P.epoch) != 0) return;
    const u8* text = P.base + P.shift;
    const int t = (int)(blockIdx.x * blockDim.x + threadIdx.x);
    u32 ns = 0, nl = 0, np = 0, centry = 0;                  // centry != 0: a short closing piece to be queued
    if (t < P.ntiles) {
        const u32 q = P.tile_q[t];
        ns = q & TQ_NS_MASK; nl = (q >> TQ_NL_SHIFT) & TQ_NL_MASK; np = P.tile_cnt[t];
    }
    u32 cn = 0, ca = 0, cslot = 0, clast = 0;
    if (np) {
        clast = P.tile_last[t];
        const u32 st = (u32)t * TT_TILE_BYTES + clast;
        cn = closing_piece_end(P, t) - st;
        ca = (u32)((long long)st - P.shift); cslot = (u32)t * TT_TILE_BYTES + np - 1;
        u32 v;
        if (piece_settled_without_merge(P, text, ca, cn, v)) { P.piece_cnt[cslot] = v; P.tile_tok[t] += 1u; cn = 0; }   // this thread is the tile's only writer here
        else if (cn <= (u32)LANE_MAX) { centry = tile_queue_entry(clast, np - 1, cn); }
        else if (cn <= (u32)TT_WARP_PIECE_MAX) P.wq[atomicAdd(&P.hdr->nwq, 1u)] = ((u64)(u32)t << 32) | tile_queue_entry(clast, np - 1, cn);
    }
    // long pieces: those inside the tile (listed by the first kernel) and a long closing piece
    const u32 nlong = nl + (cn > (u32)TT_WARP_PIECE_MAX ? 1u : 0u);
    if (nlong) {
        u32 b = atomicAdd(&P.hdr->nq_long, nlong);
        for (u32 j = 0; j < nl && j < (u32)TT_TILE_LONGCAP; j++) {
            const u32 idx = P.tile_long[(size_t)t * TT_TILE_LONGCAP + j];
            const u32 o = P.piece_off16[(size_t)t * TT_TILE_BYTES + idx], o2 = P.piece_off16[(size_t)t * TT_TILE_BYTES + idx + 1];
            P.lq[b++] = make_uint4((u32)((long long)t * TT_TILE_BYTES + o - P.shift), o2 - o, (u32)t * TT_TILE_BYTES + idx, 0u);
        }
        if (cn > (u32)TT_WARP_PIECE_MAX) P.lq[b] = make_uint4(ca, cn, cslot, 0u);
    }
    // short pieces: three lists by length (a warp later merges 32 pieces of one list at a time, a thread each, and
    // waits for the longest), one reservation per warp and list
    u64 mine = 0;                                             // four counts of 16 bits (a warp's 32 tiles hold fewer than 2^16 pieces)
    for (u32 e = 0; e < ns; e++) mine += 1ull << (16 * short_class((P.q[(size_t)t * TT_TILE_QCAP + e] >> 22) + 1));
    if (centry) mine += 1ull << (16 * short_class(cn));
    u64 pre = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const u64 v = __shfl_up_sync(FULL, pre, o); if (lane >= o) pre += v; }
    const u64 tot = __shfl_sync(FULL, pre, 31);
    u32 base[TT_SHORT_CLASSES];
#pragma unroll
    for (int c = 0; c < TT_SHORT_CLASSES; c++) {
        const u32 n = (u32)(tot >> (16 * c)) & 0xFFFFu;
        base[c] = 0;
        if (lane == 31 && n) base[c] = atomicAdd(c ? &P.hdr->nq_short_x[c - 1] : &P.hdr->nq_short, n);
    }
    pre -= mine;
#pragma unroll
    for (int c = 0; c < TT_SHORT_CLASSES; c++) base[c] = __shfl_sync(FULL, base[c], 31) + ((u32)(pre >> (16 * c)) & 0xFFFFu);
    for (u32 e = 0; e <= ns; e++) {
        if (e == ns && !centry) break;
        const u32 entry = e < ns ? P.q[(size_t)t * TT_TILE_QCAP + e] : centry;
        const int c = short_class((entry >> 22) + 1);
        const u64 x = ((u64)(u32)t << 32) | entry;
        if (c == 0) P.gq[base[0]++] = x;
        else if (c == 1) P.gq_x[0][base[1]++] = x;
        else if (c == 2) P.gq_x[1][base[2]++] = x;
        else P.gq_x[2][base[3]++] = x;
    }
}

// Long pieces of the tiles [t_lo, t_hi) (at most MERGE_THREADS of them), a whole CTA each.  Called by all threads
// of the CTA with the records of tile t_lo + tid in nl / np / last / c_end / closing_long.
__device__ void cta_long_pieces(const PieceParams& P, const u8* __restrict__ text, int t_lo, int t_hi, u32 nl, u32 np, u32 last, u32 c_end,
                                bool closing_long, u64* s_buf, u32* sc, uint4* s_long, u32* s_nlong) {
    const int tid = threadIdx.x;
    for (int k = 0; k < MERGE_THREADS && t_lo + k < t_hi; k++) {      // block-uniform; tile after tile, so that the shared list cannot overflow
        if (!__syncthreads_or(tid == k && (nl != 0 || closing_long))) continue;
        if (tid == k) {
            const int t = t_lo + k;
            u32 cnt = 0;
            for (u32 j = 0; j < nl && j < (u32)TT_TILE_LONGCAP; j++) {
                const u32 idx = P.tile_long[(size_t)t * TT_TILE_LONGCAP + j];
                const u32 o = P.piece_off16[(size_t)t * TT_TILE_BYTES + idx], o2 = P.piece_off16[(size_t)t * TT_TILE_BYTES + idx + 1];
                s_long[cnt++] = make_uint4((u32)((long long)t * TT_TILE_BYTES + o - P.shift), o2 - o, (u32)t * TT_TILE_BYTES + idx, 0u);
            }
            if (closing_long) {
                const u32 st = (u32)t * TT_TILE_BYTES + last;
                s_long[cnt++] = make_uint4((u32)((long long)st - P.shift), c_end - st, (u32)t * TT_TILE_BYTES + np - 1, 0u);
            }
            *s_nlong = cnt;
        }
        __syncthreads();
        const u32 cnt = *s_nlong;
        for (u32 e = 0; e < cnt; e++) {                               // block-uniform
            const uint4 q = s_long[e];
            __syncthreads();
            if (!piece_in_range(P, q.x, q.y, q.z, 3u)) continue;
            if (tid == 0) { u32 v = 0; sc[SCR_FLAG] = piece_settled_without_merge(P, text, q.x, q.y, v) ? 1u : 0u; sc[SCR_VALUE] = v; }
            __syncthreads();
            if (sc[SCR_FLAG]) { if (tid == 0) { P.piece_cnt[q.z] = sc[SCR_VALUE]; atomicAdd(&P.tile_tok[q.z / TT_TILE_BYTES], 1u); } continue; }
            const u32 m = cta_merge_long(text, q.x, q.y, P.tab, P.ext_id, P.stage, P.pairbuf + q.x, s_buf, sc);
            if (tid == 0) piece_done(P, q.z, m);
        }
    }
    __syncthreads();
}

// Bulk text: the last CTA of k_merge to finish sums the token counts of every group of 256 tiles for k_scatter (a
// counter cleared before the chain tells which CTA that is; nobody waits for anybody).  Called by every warp.
__device__ __forceinline__ void merge_group_totals(const PieceParams& P, u32* s_warps_done) {
    const int lane = threadIdx.x & 31;
    const u32 FULL = 0xFFFFFFFFu;
    if (P.grp_tok == nullptr) return;
    __threadfence();
    __syncwarp();
    u32 fin = 0;
    if (lane == 0 && atomicAdd(s_warps_done, 1u) == MERGE_WARPS - 1) fin = atomicAdd(&P.hdr->merge_done, 1u) == gridDim.x - 1;
    if (!__shfl_sync(FULL, fin, 0)) return;
    __threadfence();
    const int ngroups = (P.ntiles + TT_GROUP_TILES - 1) / TT_GROUP_TILES;
    for (int g = 0; g < ngroups; g++) {                               // one warp: eight loads per lane and group
        u32 sum = 0;
#pragma unroll
        for (int u = 0; u < TT_GROUP_TILES / 32; u++) { const int t = g * TT_GROUP_TILES + u * 32 + lane; if (t < P.ntiles) sum += __ldcg(&P.tile_tok[t]); }
#pragma unroll
        for (int o = 16; o; o >>= 1) sum += __shfl_xor_sync(FULL, sum, o);
        if (lane == 0) P.grp_tok[g] = sum;
    }
}

// Bulk text (k_closing has gathered the lists): long pieces a CTA each, warp-class pieces a warp each by index,
// short pieces 32 of one length class at a time by ticket, a thread each.
__device__ void merge_bulk_lists(const PieceParams& P, const u8* __restrict__ text, u64* s_buf, u32* sc, u32* s_warps_done) {
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const u32 FULL = 0xFFFFFFFFu;
    const u32 nl = P.hdr->nq_long, nw = P.hdr->nwq, ns = P.hdr->nq_short;
    for (u32 e = blockIdx.x; e < nl; e += gridDim.x) {                // block-uniform
        const uint4 q = P.lq[e];
        __syncthreads();
        if (!piece_in_range(P, q.x, q.y, q.z, 3u)) continue;
        const u32 m = cta_merge_long(text, q.x, q.y, P.tab, P.ext_id, P.stage, P.pairbuf + q.x, s_buf, sc);
        if (tid == 0) piece_done(P, q.z, m);
    }
    if (nl > blockIdx.x) __syncthreads();
    u64* wbuf = s_buf + wid * WARP_SMEM_WORDS;
    const u32 W = gridDim.x * MERGE_WARPS, gw = (u32)wid * gridDim.x + blockIdx.x;
    for (u32 j = gw; j < nw; j += W) {                                // bounded by the list length
        const u64 x = P.wq[j];
        const u32 t = (u32)(x >> 32), e = (u32)x;
        warp_merge_piece(P, text, (u32)((long long)t * TT_TILE_BYTES + (e & 2047u) - P.shift), (e >> 22) + 1, t * TT_TILE_BYTES + ((e >> 11) & 2047u), wbuf, lane);
    }
    u32* const tok = reinterpret_cast<u32*>(wbuf);
    // tickets: 32 pieces of one list each, the list of the longest pieces first
    u32 cnts[TT_SHORT_CLASSES], nb[TT_SHORT_CLASSES], nball = 0;
#pragma unroll
    for (int c = 0; c < TT_SHORT_CLASSES; c++) { cnts[c] = c ? P.hdr->nq_short_x[c - 1] : ns; nb[c] = (cnts[c] + LANE_SLOTS - 1) / LANE_SLOTS; nball += nb[c]; }
    for (;;) {                                                        // bounded by the number of tickets
        u32 tk = 0;
        if (lane == 0) tk = atomicAdd(&P.hdr->t_short, 1u);
        tk = __shfl_sync(FULL, tk, 0);
        if (tk >= nball) break;
        const u64* list = P.gq; u32 cnt = 0, e0 = 0;
        {
            u32 r = tk;
            bool found = false;
#pragma unroll
            for (int c = TT_SHORT_CLASSES - 1; c >= 0; c--) {
                if (!found && r < nb[c]) { list = c ? P.gq_x[c - 1] : P.gq; cnt = cnts[c]; e0 = r * LANE_SLOTS; found = true; }
                if (!found) r -= nb[c];
            }
        }
        if (e0 + lane < cnt) {
            const u64 x = list[e0 + lane];
            const u32 t = (u32)(x >> 32), e = (u32)x;
            const u32 a = (u32)((long long)t * TT_TILE_BYTES + (e & 2047u) - P.shift), n = (e >> 22) + 1, slot = t * TT_TILE_BYTES + ((e >> 11) & 2047u);
            if (!piece_in_range(P, a, n, slot, 4u) || n < 2 || n > (u32)LANE_MAX) hdr_selfcheck_failed(P.hdr, P.epoch, 5u, a, n, slot, e0);
            else {
                const u32 m = lane_merge(tok, tok + LANE_SLOTS * LANE_MAX, lane, text, a, n, P.tab, P.ext_id, P.stage);
                piece_done(P, slot, m);
            }
        }
        __syncwarp();
    }
    merge_group_totals(P, s_warps_done);
}

// The merge kernel of bulk text (more tiles than a request's job search covers): works off the lists k_closing built.
__global__ void __launch_bounds__(MERGE_THREADS, MERGE_CTAS_PER_SM)
k_merge_bulk(const __grid_constant__ PieceParams P) {
    extern __shared__ __align__(16) u64 s_buf[];              // MERGE_SMEM_BYTES
    __shared__ u32 sc[SCR_WORDS];
    __shared__ u32 s_warps_done;
    cudaTriggerProgrammaticLaunchCompletion();               // k_scatter may be placed; it waits for this grid's memory itself
    grid_prefetch_l2(P.tab.slots, ((size_t)P.tab.mask + 1) * 2 * sizeof(uint4));
    grid_prefetch_l2(P.tab.bytepair, 65536 * sizeof(u64));
    if (threadIdx.x == 0) s_warps_done = 0;
    cudaGridDependencySynchronize();                         // k_closing's lists are complete from here on
    __syncthreads();
    if (hdr_status(P.hdr, P.epoch) != 0) return;
    merge_bulk_lists(P, P.base + P.shift, s_buf, sc, &s_warps_done);
}

__global__ void __launch_bounds__(MERGE_THREADS, MERGE_CTAS_PER_SM)
k_merge(const __grid_constant__ PieceParams P) {
    extern __shared__ __align__(16) u64 s_buf[];              // MERGE_SMEM_BYTES
    __shared__ u32 sc[SCR_WORDS];
    __shared__ uint4 s_long[TT_TILE_LONGCAP + 2];             // the long pieces of one tile
    __shared__ u32 s_nlong;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const u32 FULL = 0xFFFFFFFFu;
    cudaTriggerProgrammaticLaunchCompletion();               // k_scatter may be placed; it waits for this grid's memory itself
    grid_prefetch_l2(P.tab.slots, ((size_t)P.tab.mask + 1) * 2 * sizeof(uint4));
    grid_prefetch_l2(P.tab.bytepair, 65536 * sizeof(u64));
    cudaGridDependencySynchronize();                         // the first kernel's per-tile records are complete from here on
    if (hdr_status(P.hdr, P.epoch) != 0) return;
    const u8* text = P.base + P.shift;
    // ---- records of this CTA's share of the tiles (long pieces, a whole CTA each; a request settles them after
    // its short pieces, bulk text before); the loads go out next to those of the job search below
    const int per = (P.ntiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int t_lo = (int)blockIdx.x * per, t_hi = min(P.ntiles, t_lo + per);
    u32 a_nl = 0, a_np = 0, a_last = 0, a_next = TT_NONE;
    {
        const int t = t_lo + tid;
        if (t < t_hi) {
            a_nl = (P.tile_q[t] >> TQ_NL_SHIFT) & TQ_NL_MASK; a_np = P.tile_cnt[t]; a_last = P.tile_last[t];
            if (t + 1 < P.ntiles) a_next = P.tile_first[t + 1];
        }
    }
    u64* wbuf = s_buf + wid * WARP_SMEM_WORDS;
    const u32 W = gridDim.x * MERGE_WARPS, gw = (u32)wid * gridDim.x + blockIdx.x;   // numbered across the CTAs first
    const bool big = false;                                       // (bulk text took the lists above)
    // job search of a request: every lane sums the counts of a stretch of tiles, kept as 16 sums of `unit` tiles
    // (short pieces in the low half, warp-class pieces in the high half of a word)
    const int unit = (P.ntiles + 511) / 512;                      // 1..4 tiles per register
    const int tb = lane * 16 * unit;
    u32 part[16];
    u32 my_s = 0, my_w = 0;
    if (!big) {
        if (unit == 1) {                                          // up to 512 tiles: sixteen counts per lane, four vector loads
            const uint4* src = reinterpret_cast<const uint4*>(P.tile_q + tb);
            uint4 v[4];
#pragma unroll
            for (int g = 0; g < 4; g++) v[g] = tb + 4 * g < P.ntiles ? src[g] : make_uint4(0, 0, 0, 0);
#pragma unroll
            for (int g = 0; g < 16; g++) {
                const uint4 x = v[g >> 2];
                const u32 q = (g & 3) == 0 ? x.x : (g & 3) == 1 ? x.y : (g & 3) == 2 ? x.z : x.w;
                part[g] = tb + g < P.ntiles ? (q & TQ_NS_MASK) | (((q >> TQ_NW_SHIFT) & TQ_NW_MASK) << 16) : 0u;
            }
        } else {
#pragma unroll
            for (int g = 0; g < 16; g++) {
                u32 s1 = 0;
                for (int u = 0; u < unit; u++) {
                    const int t = tb + g * unit + u;
                    if (t < P.ntiles) { const u32 q = P.tile_q[t]; s1 += (q & TQ_NS_MASK) | (((q >> TQ_NW_SHIFT) & TQ_NW_MASK) << 16); }
                }
                part[g] = s1;
            }
        }
#pragma unroll
        for (int g = 0; g < 16; g++) { my_s += part[g] & 0xFFFFu; my_w += part[g] >> 16; }
    }
    // the closing piece of tile t_lo + tid: is it long?
    bool closing_long = false;
    u32 c_end = 0;
    if (a_np) {
        const int t = t_lo + tid;
        c_end = (t + 1 >= P.ntiles) ? (u32)P.hi : a_next != TT_NONE ? (u32)(t + 1) * TT_TILE_BYTES + a_next : closing_piece_end(P, t);
        closing_long = c_end - ((u32)t * TT_TILE_BYTES + a_last) > (u32)TT_WARP_PIECE_MAX;
    }
    bool tickets = big;                                           // short pieces by tickets (bulk) or job by job (a request)
    if (!big) {
        u32 bs = my_s, bw = my_w;                                     // exclusive prefixes over the lanes
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const u32 x = __shfl_up_sync(FULL, bs, o), y = __shfl_up_sync(FULL, bw, o);
            if (lane >= o) { bs += x; bw += y; }
        }
        const u32 NS = __shfl_sync(FULL, bs, 31), NW = __shfl_sync(FULL, bw, 31), NT = (u32)P.ntiles;
        bs -= my_s; bw -= my_w;
#ifndef TT_SHORT_WARP_FACTOR
#define TT_SHORT_WARP_FACTOR 12u
#endif
        // Measured crossover (1 M to 8 M chars of Unicode-heavy prose, 15 K to 120 K unsettled pieces): a warp per piece
        // wins up to about 17 pieces per warp of the grid.
        tickets = NS + NT > TT_SHORT_WARP_FACTOR * W;
        const u32 J = tickets ? NW : NW + NT + NS;                    // with tickets only the warp-class pieces go job by job
        for (u32 j = gw; j < J; j += W) {                             // bounded by the number of jobs
            u32 a, n, slot;
            if (j >= NW && j < NW + NT) {                             // the closing piece of tile j - NW
                const int t = (int)(j - NW);
                const u32 np = P.tile_cnt[t];
                if (np == 0) continue;
                const u32 st = (u32)t * TT_TILE_BYTES + P.tile_last[t];
                n = closing_piece_end(P, t) - st;
                if (n > (u32)TT_WARP_PIECE_MAX) continue;             // settled by a CTA below
                a = (u32)((long long)st - P.shift); slot = (u32)t * TT_TILE_BYTES + np - 1;
                u32 v;
                if (piece_settled_without_merge(P, text, a, n, v)) {  // every lane computes the same
                    if (lane == 0) { P.piece_cnt[slot] = v; atomicAdd(&P.tile_tok[t], 1u); }
                    continue;
                }
            } else {
                // the k-th queued piece of its class: the lane whose stretch holds it finds the tile
                const bool wclass = j < NW;
                const u32 k = wclass ? j : j - NW - NT;
                const int sh = wclass ? 16 : 0;
                const u32 owner = 31u - (u32)__clz(__ballot_sync(FULL, (wclass ? bw : bs) <= k) | 1u);
                u32 found = 0;                                        // tile << 11 | rank within the tile
                if ((u32)lane == owner) {
                    u32 r = k - (wclass ? bw : bs);
                    int g = 0;
#pragma unroll
                    for (int gg = 0; gg < 15; gg++) {
                        const u32 c = (part[gg] >> sh) & 0xFFFFu;
                        if (g == gg && r >= c) { r -= c; g = gg + 1; }
                    }
                    int t = tb + g * unit;
                    for (int u = 0; u + 1 < unit; u++) {
                        const u32 q = t < P.ntiles ? P.tile_q[t] : 0u;
                        const u32 c = wclass ? (q >> TQ_NW_SHIFT) & TQ_NW_MASK : q & TQ_NS_MASK;
                        if (r < c) break;
                        r -= c; t++;
                    }
                    found = ((u32)t << 11) | r;
                }
                found = __shfl_sync(FULL, found, owner);
                const u32 t = found >> 11, r = found & 2047u;
                const u32 e = P.q[(size_t)t * TT_TILE_QCAP + (wclass ? (u32)TT_TILE_QCAP - 1 - r : r)];
                n = (e >> 22) + 1;
                a = (u32)((long long)t * TT_TILE_BYTES + (e & 2047u) - P.shift); slot = t * TT_TILE_BYTES + ((e >> 11) & 2047u);
            }
            warp_merge_piece(P, text, a, n, slot, wbuf, lane);
        }
        if (!tickets) {
            // the request's long pieces, once every warp of the CTA is through with its short ones
            if (__syncthreads_or(a_nl != 0 || closing_long))
                cta_long_pieces(P, text, t_lo, t_hi, a_nl, a_np, a_last, c_end, closing_long, s_buf, sc, s_long, &s_nlong);
            return;
        }
    }
    for (int t0 = t_lo; t0 < t_hi; t0 += MERGE_THREADS) {            // block-uniform; shares beyond MERGE_THREADS tiles reload their records
        if (t0 != t_lo) {
            const int t = t0 + tid;
            a_nl = 0; a_np = 0; a_last = 0; c_end = 0; closing_long = false;
            if (t < t_hi) {
                a_nl = (P.tile_q[t] >> TQ_NL_SHIFT) & TQ_NL_MASK; a_np = P.tile_cnt[t]; a_last = P.tile_last[t];
                if (a_np) { c_end = closing_piece_end(P, t); closing_long = c_end - ((u32)t * TT_TILE_BYTES + a_last) > (u32)TT_WARP_PIECE_MAX; }
            }
        }
        if (__syncthreads_or(a_nl != 0 || closing_long))
            cta_long_pieces(P, text, t0, t_hi, a_nl, a_np, a_last, c_end, closing_long, s_buf, sc, s_long, &s_nlong);
    }
    // ---- tickets: a tile each; its short pieces (queued ones, then its closing piece if that is short) wait in the
    // lanes until 32 of them are together, so that every step of the thread-per-piece merge is full
    {
        u32* const tok = reinterpret_cast<u32*>(wbuf);
        const u32 ntick = (u32)P.ntiles;
        u32 pa = 0, pn = 0, pslot = 0, pend = 0;                      // lanes below `pend` hold a short piece that waits for a full step
        for (;;) {                                                    // bounded by the number of tickets
            u32 t = 0;
            if (lane == 0) t = atomicAdd(&P.hdr->t_tiles, 1u);
            t = __shfl_sync(FULL, t, 0);
            const bool last_round = t >= ntick;
            u32 ns = 0, ca = 0, cn = 0, cslot = 0;                    // cn == 0: no closing piece left to merge
            if (!last_round) {                                        // warp-uniform; every lane computes the same
                const u32 q = P.tile_q[t], np = P.tile_cnt[t], last = P.tile_last[t];
                const u32 nf = t + 1 < ntick ? P.tile_first[t + 1] : TT_NONE;
                ns = q & TQ_NS_MASK;
                if (np) {
                    const u32 st = t * TT_TILE_BYTES + last;
                    cn = (t + 1 >= ntick ? (u32)P.hi : nf != TT_NONE ? (t + 1) * TT_TILE_BYTES + nf : closing_piece_end(P, (int)t)) - st;
                    ca = (u32)((long long)st - P.shift); cslot = t * TT_TILE_BYTES + np - 1;
                    u32 v;
                    if (cn > (u32)TT_WARP_PIECE_MAX) cn = 0;          // settled by a CTA above
                    else if (piece_settled_without_merge(P, text, ca, cn, v)) { if (lane == 0) { P.piece_cnt[cslot] = v; atomicAdd(&P.tile_tok[t], 1u); } cn = 0; }
                    else if (cn > (u32)LANE_MAX) { warp_merge_piece(P, text, ca, cn, cslot, wbuf, lane); cn = 0; }
                }
            }
            const u32 nj = ns + (cn ? 1u : 0u);
            u32 e0 = 0;                                               // new pieces handed to lanes so far
            for (;;) {                                                // warp-uniform; bounded by nj / 32 + 2
                const u32 left = nj - e0;
                const bool run = pend + left >= 32u || (last_round && pend != 0);
                const u32 take = min(32u - pend, left);               // lanes pend .. pend + take - 1 take new pieces
                const u32 e = e0 + ((u32)lane - pend);
                if ((u32)lane >= pend && (u32)lane - pend < take) {
                    if (e < ns) {
                        const u32 qe = P.q[(size_t)t * TT_TILE_QCAP + e];
                        pn = (qe >> 22) + 1;
                        pa = (u32)((long long)t * TT_TILE_BYTES + (qe & 2047u) - P.shift); pslot = t * TT_TILE_BYTES + ((qe >> 11) & 2047u);
                    } else { pa = ca; pn = cn; pslot = cslot; }
                }
                e0 += take; pend += take;
                if (!run) break;
                if ((u32)lane < pend) {
                    if (!piece_in_range(P, pa, pn, pslot, 4u) || pn < 2 || pn > (u32)LANE_MAX) hdr_selfcheck_failed(P.hdr, P.epoch, 5u, pa, pn, pslot, e);
                    else {
                        const u32 m = lane_merge(tok, tok + LANE_SLOTS * LANE_MAX, lane, text, pa, pn, P.tab, P.ext_id, P.stage);
                        piece_done(P, pslot, m);
                    }
                }
                __syncwarp();
                pend = 0;
            }
            if (last_round) break;
        }
    }
}

// ---- K5: coalesced scatter of the staged ids, one text tile per CTA iteration ---------------------------------
// Also writes the token offset of every document that starts in the tile (batch calls).
struct ScatterParams {
    long long shift, hi;
    int ntiles;
    const u32* tile_cnt;
    const u32* tile_tok;       // tokens per tile
    const u32* grp_tok;        // bulk text: tokens per group of TT_GROUP_TILES tiles, else null
    const u16* piece_off16;
    unsigned long long ids_cap;
    const u32* piece_cnt;
    const int32_t* stage;
    TTHeader* hdr;
    unsigned long long epoch;
    int32_t* ids_out;
    long long* count_out;
    int32_t* status_out;
    const u32* docmask;        // batch: bit per byte of document starts, else null
    const long long* doc_off;  // batch: n_docs + 1 offsets
    int n_docs;
    long long* ids_off_out;    // batch: n_docs + 1 token offsets
};

constexpr int SCATTER_STAGE_IDS = 2048;                   // ids of one work item that are put together in shared memory
__global__ void __launch_bounds__(BPE_THREADS)
k_scatter(const ScatterParams P) {
    __shared__ u32 sc[SCR_WORDS];
    __shared__ u32 s_big[TT_TILE_BYTES / 8][3];
    __shared__ u32 s_nbig;
    __shared__ u32 s_np[BPE_THREADS];                         // pieces of the next tiles of this CTA's range
    __shared__ int32_t s_out[SCATTER_STAGE_IDS];              // the ids of one item on their way out
    __shared__ unsigned long long s_sum[66];
    const int tid = threadIdx.x;
    cudaGridDependencySynchronize();                         // k_merge's (and with it the first kernel's) results are complete from here on
    // Each CTA takes a contiguous range of tiles.  Tokens before its first tile: a request's CTAs sum the counts of
    // all tiles themselves; for bulk text k_merge has left the totals of groups of tiles, so a CTA adds the whole
    // groups before its range and the tiles of its own group before it.  The grand total gives the count and the
    // capacity check, which every CTA makes for itself.
    const int per = (P.ntiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int tile_lo = (int)blockIdx.x * per, tile_hi = min(P.ntiles, tile_lo + per);
    unsigned long long before = 0, total = 0;
    if (P.grp_tok == nullptr) {
        for (int t0 = 0; t0 < P.ntiles; t0 += BPE_THREADS * 4) {
            u32 x[4];
#pragma unroll
            for (int u = 0; u < 4; u++) { const int t = t0 + u * BPE_THREADS + tid; x[u] = t < P.ntiles ? P.tile_tok[t] : 0u; }
#pragma unroll
            for (int u = 0; u < 4; u++) { total += x[u]; if (t0 + u * BPE_THREADS + tid < tile_lo) before += x[u]; }
        }
    } else {
        const int ngroups = (P.ntiles + TT_GROUP_TILES - 1) / TT_GROUP_TILES, g_lo = tile_lo / TT_GROUP_TILES;
        for (int g = tid; g < ngroups; g += BPE_THREADS) { const u32 x = P.grp_tok[g]; total += x; if (g < g_lo) before += x; }
        for (int t = g_lo * TT_GROUP_TILES + tid; t < tile_lo; t += BPE_THREADS) before += P.tile_tok[t];
    }
    cta_sum2_u64(before, total, s_sum);
    int status = hdr_status(P.hdr, P.epoch);
    if (status == 0 && total > P.ids_cap) status = 5;          // TT_ERR_CAPACITY
    if (blockIdx.x == 0 && tid == 0) {
        if (P.status_out) *P.status_out = status;
        if (P.count_out) *P.count_out = status ? 0 : (long long)total;
    }
    if (status != 0) {
        if (P.ids_off_out)
            for (long long d = (long long)blockIdx.x * blockDim.x + tid; d <= P.n_docs; d += (long long)gridDim.x * blockDim.x) P.ids_off_out[d] = 0;
        return;
    }
    if (P.ids_off_out && blockIdx.x == 0) {
        // documents that start at the very end of the text (empty trailing documents) and the total
        const long long len = P.hi - P.shift;
        for (int d = P.n_docs - tid; d >= 0 && P.doc_off[d] >= len; d -= blockDim.x) P.ids_off_out[d] = (long long)total;
    }
    // Work items: (tile, block of 512 of its pieces), two neighbouring pieces per thread.  The loads of the next item
    // (piece values and offsets) go out before the current one is scanned and written, so that the chain
    // "count of the tile -> its piece values -> scan -> staged ids" of one tile overlaps with the next tile's.
    u32 carry = (u32)before;
    for (int tc = tile_lo; tc < tile_hi; tc += BPE_THREADS) {         // block-uniform
        const int nk = min(BPE_THREADS, tile_hi - tc);
        __syncthreads();
        if (tid < nk) s_np[tid] = P.tile_cnt[tc + tid];
        if (tid == 0) s_nbig = 0;
        __syncthreads();
        int k = 0;
        u32 b = 0;
        while (k < nk && s_np[k] == 0) k++;
        uint2 v = make_uint2(0, 0);
        u32 o2 = 0;
        if (k < nk) {
            const size_t p0 = (size_t)(tc + k) * TT_TILE_BYTES;
            const u32 i0 = 2 * (u32)tid;
            if (i0 < s_np[k]) { v = *reinterpret_cast<const uint2*>(P.piece_cnt + p0 + i0); o2 = *reinterpret_cast<const u32*>(P.piece_off16 + p0 + i0); }
        }
        while (k < nk) {                                              // block-uniform
            // the item after this one
            int k2 = k;
            u32 b2 = b + 2 * BPE_THREADS;
            if (b2 >= s_np[k2]) { b2 = 0; k2++; while (k2 < nk && s_np[k2] == 0) k2++; }
            uint2 vn = make_uint2(0, 0);
            u32 on = 0;
            if (k2 < nk) {
                const size_t q0 = (size_t)(tc + k2) * TT_TILE_BYTES;
                const u32 j0 = b2 + 2 * (u32)tid;
                if (j0 < s_np[k2]) { vn = *reinterpret_cast<const uint2*>(P.piece_cnt + q0 + j0); on = *reinterpret_cast<const u32*>(P.piece_off16 + q0 + j0); }
            }
            // this item
            const int tile = tc + k;
            const u32 np = s_np[k], i0 = b + 2 * (u32)tid;
            const long long t0 = (long long)tile * TT_TILE_BYTES - P.shift;  // text offset of the tile start
            const int32_t x0 = i0 < np ? (int32_t)v.x : 0, x1 = i0 + 1 < np ? (int32_t)v.y : 0;   // an id, or minus the staged count
            const u32 c0 = i0 < np ? (x0 >= 0 ? 1u : (u32)(-x0)) : 0u, c1 = i0 + 1 < np ? (x1 >= 0 ? 1u : (u32)(-x1)) : 0u;
            u32 tot;
            const u32 d0 = carry + cta_excl_sum_scan(c0 + c1, sc, &tot);
            // An item without pieces of more than eight tokens (nearly all) is put together in shared memory and leaves in
            // whole lines, every thread writing consecutive words: the output may be mapped host memory, where a warp that
            // writes every other word costs a bus transaction per word.
            const bool staged = !__syncthreads_or(c0 > 8 || c1 > 8) && tot <= (u32)SCATTER_STAGE_IDS;
#pragma unroll
            for (int h = 0; h < 2; h++) {
                const u32 i = i0 + h, c = h ? c1 : c0, dst = h ? d0 + c0 : d0, off = h ? o2 >> 16 : o2 & 0xFFFFu;
                const int32_t x = h ? x1 : x0;
                if (i >= np) continue;
                if ((unsigned long long)dst + c > total || (x < 0 && t0 + off + c > P.hi - P.shift)) { hdr_selfcheck_failed(P.hdr, P.epoch, 6u, (u32)tile, i, (u32)x, dst); continue; }
                const u32 src = (u32)(t0 + off);
                int32_t* const out = staged ? s_out - carry : P.ids_out;             // same index either way
                if (x >= 0) out[dst] = x;
                else if (c <= 8) { for (u32 kk = 0; kk < c; kk++) out[dst + kk] = P.stage[src + kk]; }
                else {
                    const u32 slot = atomicAdd(&s_nbig, 1u);
                    if (slot < TT_TILE_BYTES / 8) { s_big[slot][0] = src; s_big[slot][1] = dst; s_big[slot][2] = c; }
                }
                if (P.docmask) {
                    const long long g = (long long)tile * TT_TILE_BYTES + off;
                    if ((P.docmask[g >> 5] >> (g & 31)) & 1) {
                        // every document that starts at this byte (empty ones included) gets this token offset
                        const long long want = g - P.shift;
                        int lo = 0, hi2 = P.n_docs;
                        while (lo < hi2) { int mid = (lo + hi2) >> 1; if (P.doc_off[mid] < want) lo = mid + 1; else hi2 = mid; }
                        for (int d = lo; d <= P.n_docs && P.doc_off[d] == want; d++) P.ids_off_out[d] = dst;
                    }
                }
            }
            if (staged) {                                             // block-uniform
                __syncthreads();
                for (u32 kk = tid; kk < tot; kk += BPE_THREADS) P.ids_out[carry + kk] = s_out[kk];
            }
            carry += tot;
            __syncthreads();
            const u32 nbig = min(s_nbig, (u32)(TT_TILE_BYTES / 8));
            if (nbig) {                                               // block-uniform: pieces of more than 8 tokens, copied by the whole CTA
                for (u32 e = 0; e < nbig; e++) {
                    const u32 src = s_big[e][0], d2 = s_big[e][1], cc = s_big[e][2];
                    for (u32 kk = tid; kk < cc; kk += BPE_THREADS) P.ids_out[d2 + kk] = P.stage[src + kk];
                }
                __syncthreads();
                if (tid == 0) s_nbig = 0;
            }
            k = k2; b = b2; v = vn; o2 = on;
        }
    }
}

// ---- K5 for bulk text: a warp per tile, no barrier after the prologue -----------------------------------------
// Each CTA takes a contiguous range of tiles, its warps every eighth tile of it.  A warp knows where its tile's ids
// go from the token counts of the tiles before it (group totals, then tile counts), scans the tile's pieces 128 at
// a time (four neighbouring pieces per lane, one 16-byte load) with warp shuffles, and copies pieces of more than
// eight tokens with all its lanes.
__global__ void __launch_bounds__(BPE_THREADS)
k_scatter_bulk(const ScatterParams P) {
    __shared__ unsigned long long s_sum[66];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const u32 FULL = 0xFFFFFFFFu;
    cudaGridDependencySynchronize();                         // k_merge_bulk's (and with it the kernels' before it) results are complete
    const int per = (P.ntiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int tile_lo = (int)blockIdx.x * per, tile_hi = min(P.ntiles, tile_lo + per);
    unsigned long long before = 0, total = 0;
    {
        const int ngroups = (P.ntiles + TT_GROUP_TILES - 1) / TT_GROUP_TILES, g_lo = tile_lo / TT_GROUP_TILES;
        for (int g = tid; g < ngroups; g += BPE_THREADS) { const u32 x = P.grp_tok[g]; total += x; if (g < g_lo) before += x; }
        for (int t = g_lo * TT_GROUP_TILES + tid; t < tile_lo; t += BPE_THREADS) before += P.tile_tok[t];
    }
    cta_sum2_u64(before, total, s_sum);
    int status = hdr_status(P.hdr, P.epoch);
    if (status == 0 && total > P.ids_cap) status = 5;          // TT_ERR_CAPACITY
    if (blockIdx.x == 0 && tid == 0) {
        if (P.status_out) *P.status_out = status;
        if (P.count_out) *P.count_out = status ? 0 : (long long)total;
    }
    if (status != 0) {
        if (P.ids_off_out)
            for (long long d = (long long)blockIdx.x * blockDim.x + tid; d <= P.n_docs; d += (long long)gridDim.x * blockDim.x) P.ids_off_out[d] = 0;
        return;
    }
    if (P.ids_off_out && blockIdx.x == 0) {
        const long long len = P.hi - P.shift;
        for (int d = P.n_docs - tid; d >= 0 && P.doc_off[d] >= len; d -= blockDim.x) P.ids_off_out[d] = (long long)total;
    }
    // tokens of the tiles of this CTA's range before the warp's first tile
    u32 carry = (u32)before;
    {
        u32 x = (lane < wid && tile_lo + lane < tile_hi) ? P.tile_tok[tile_lo + lane] : 0u;
#pragma unroll
        for (int o = 16; o; o >>= 1) x += __shfl_xor_sync(FULL, x, o);
        carry += x;
    }
    for (int tile = tile_lo + wid; tile < tile_hi; tile += BPE_WARPS) {   // warp-uniform
        const u32 np = P.tile_cnt[tile];
        // the seven tiles between this one and the warp's next
        u32 skip = (lane >= 1 && lane < BPE_WARPS && tile + lane < tile_hi) ? P.tile_tok[tile + lane] : 0u;
        const size_t p0 = (size_t)tile * TT_TILE_BYTES;
        const long long t0 = (long long)tile * TT_TILE_BYTES - P.shift;      // text offset of the tile start
        // does any document start in this tile?  (few tiles: the pieces of the others need not look)
        bool tile_has_doc = false;
        if (P.docmask) {
            const size_t wi = (size_t)tile * (TT_TILE_BYTES / 32) + 2 * lane, nwords = (size_t)(P.hi >> 5) + 4;   // (the mask's cleared extent)
            uint2 dm = make_uint2(0, 0);
            if (wi + 1 < nwords) dm = *reinterpret_cast<const uint2*>(P.docmask + wi);
            else if (wi < nwords) dm.x = P.docmask[wi];
            tile_has_doc = __any_sync(FULL, (dm.x | dm.y) != 0);
        }
        u32 run = carry;
        uint4 v = make_uint4(0, 0, 0, 0);
        uint2 o4 = make_uint2(0, 0);
        if (4u * lane < np) { v = *reinterpret_cast<const uint4*>(P.piece_cnt + p0 + 4 * lane); o4 = *reinterpret_cast<const uint2*>(P.piece_off16 + p0 + 4 * lane); }
        for (u32 b = 0; b < np; b += 128) {                               // warp-uniform
            // the next 128 pieces
            uint4 vn = make_uint4(0, 0, 0, 0);
            uint2 on = make_uint2(0, 0);
            const u32 j0 = b + 128 + 4 * lane;
            if (j0 < np) { vn = *reinterpret_cast<const uint4*>(P.piece_cnt + p0 + j0); on = *reinterpret_cast<const uint2*>(P.piece_off16 + p0 + j0); }
            const u32 i0 = b + 4 * lane;
            const int32_t x[4] = {(int32_t)v.x, (int32_t)v.y, (int32_t)v.z, (int32_t)v.w};
            const u32 off[4] = {o4.x & 0xFFFFu, o4.x >> 16, o4.y & 0xFFFFu, o4.y >> 16};
            u32 c[4], mine = 0;
#pragma unroll
            for (int h = 0; h < 4; h++) { c[h] = i0 + h < np ? (x[h] >= 0 ? 1u : (u32)(-x[h])) : 0u; mine += c[h]; }
            u32 inc = mine;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) { const u32 y = __shfl_up_sync(FULL, inc, o); if (lane >= o) inc += y; }
            const u32 tot = __shfl_sync(FULL, inc, 31);
            u32 dst = run + inc - mine;
            u32 bigmask = 0;                                              // which of my four pieces have more than eight tokens
#pragma unroll
            for (int h = 0; h < 4; h++) {
                const u32 i = i0 + h;
                if (i < np) {
                    const u32 src = (u32)(t0 + off[h]);
                    if ((unsigned long long)dst + c[h] > total || (x[h] < 0 && t0 + off[h] + c[h] > P.hi - P.shift)) hdr_selfcheck_failed(P.hdr, P.epoch, 7u, (u32)tile, i, (u32)x[h], dst);
                    else if (x[h] >= 0) P.ids_out[dst] = x[h];
                    else if (c[h] <= 8) { for (u32 kk = 0; kk < c[h]; kk++) P.ids_out[dst + kk] = P.stage[src + kk]; }
                    else bigmask |= 1u << h;
                    if (tile_has_doc) {
                        const long long g = (long long)tile * TT_TILE_BYTES + off[h];
                        if ((P.docmask[g >> 5] >> (g & 31)) & 1) {
                            // every document that starts at this byte (empty ones included) gets this token offset
                            const long long want = g - P.shift;
                            int lo = 0, hi2 = P.n_docs;
                            while (lo < hi2) { int mid = (lo + hi2) >> 1; if (P.doc_off[mid] < want) lo = mid + 1; else hi2 = mid; }
                            for (int d = lo; d <= P.n_docs && P.doc_off[d] == want; d++) P.ids_off_out[d] = dst;
                        }
                    }
                }
                dst += c[h];
            }
            // pieces of more than eight tokens: copied by the whole warp, one after the other
#pragma unroll
            for (int h = 0; h < 4; h++) {
                for (u32 m = __ballot_sync(FULL, (bigmask >> h) & 1); m; m &= m - 1) {     // warp-uniform
                    const int l = __ffs(m) - 1;
                    u32 d2 = run + inc - mine;
#pragma unroll
                    for (int g = 0; g < 4; g++) if (g < h) d2 += c[g];
                    const u32 src = __shfl_sync(FULL, (u32)(t0 + off[h]), l), dd = __shfl_sync(FULL, d2, l), cc = __shfl_sync(FULL, c[h], l);
                    for (u32 kk = lane; kk < cc; kk += 32) P.ids_out[dd + kk] = P.stage[src + kk];
                }
            }
            run += tot;
            v = vn; o4 = on;
        }
#pragma unroll
        for (int o = 16; o; o >>= 1) skip += __shfl_xor_sync(FULL, skip, o);
        carry = run + skip;
    }
}

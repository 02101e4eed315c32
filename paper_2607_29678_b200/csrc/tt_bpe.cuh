// Steps K4 and K5: byte-level BPE per piece, token counts and scatter of the IDs.
//
// Paper Sec. 4.2: every piece is encoded independently; merge ranks and vocabulary entries live in
// GPU hash tables; a round's minimum rank identifies one pair value, merging all its leftmost
// non-overlapping occurrences equals iterated single merges, and only pairs next to a completed
// merge need to be probed again.  Work is dispatched by piece length and difficulty:
//   * k_lookup: a thread per piece looks the whole piece up as a vocabulary entry (one 32-byte probe); pieces
//     that are not a single entry are appended to global queues by length class;
//   * k_merge: every warp of the GPU draws from those queues -- a warp per piece (<= 32 bytes: tokens in
//     registers, candidates as ballot masks; <= 256 bytes: several tokens per lane, compaction through shared
//     memory), or, where the call has many pieces of <= 32 bytes, 32 of them at once, a thread per piece
//     (lane_merge); longer pieces are merged by a whole CTA (cta_merge_long: state in shared memory, or in
//     global scratch while the piece still has more than 4,096 tokens).
// Token ids inside the kernels are "internal": byte b -> b, result of the merge of rank r -> 256 + r;
// the caller's ids are looked up when the tokens are staged.
#pragma once
#include "tt_common.cuh"

// ---- pair table: (left, right) -> rank ---------------------------------------------------------------
// Buckets of four 8-byte slots (one 32-byte sector); slot = (left << 38) | (right << 20) | rank.
// A key lives in its home bucket or, if that is full, in the following ones; a bucket with a free
// slot ends the search.  Sized for at most one key per bucket on average.
struct PairTable {
    const u64* slots;     // 4 * (mask + 1) slots
    const u32* bytepair;  // rank of the pair (byte a, byte b) at [a << 8 | b], TT_RANK_INF if none: a piece's first probes
    u32 mask;             // number of buckets - 1 (power of two)
    u32 shift;            // 32 - log2(number of buckets)
};
TT_HD u32 pair_bucket(u64 key, u32 shift) {
    const u32 x = ((u32)key ^ ((u32)(key >> 32) * 0x9E3779B1u)) * 0x85EBCA6Bu;
    return (x ^ (x >> 15)) * 0xC2B2AE35u >> shift;
}

__device__ __forceinline__ u32 pair_probe(const PairTable& t, u32 a, u32 b) {
    const u64 key = ((u64)a << TT_ID_BITS) | b;
    u32 h = pair_bucket(key, t.shift);
    for (u32 n = 0; n <= t.mask; n++) {               // bounded by the number of buckets
        const uint4* bp = reinterpret_cast<const uint4*>(t.slots + 4 * (size_t)h);
        const uint4 x = __ldg(bp), y = __ldg(bp + 1);
        const u64 s0 = ((u64)x.y << 32) | x.x, s1 = ((u64)x.w << 32) | x.z, s2 = ((u64)y.y << 32) | y.x, s3 = ((u64)y.w << 32) | y.z;
        if ((s0 >> 20) == key) return (u32)(s0 & 0xFFFFFu);
        if ((s1 >> 20) == key) return (u32)(s1 & 0xFFFFFu);
        if ((s2 >> 20) == key) return (u32)(s2 & 0xFFFFFu);
        if ((s3 >> 20) == key) return (u32)(s3 & 0xFFFFFu);
        if (s3 == TT_SLOT_EMPTY) return TT_RANK_INF;  // slots fill from the front: a free last slot ends the chain
        h = (h + 1) & t.mask;
    }
    return TT_RANK_INF;
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
// returns what the merge loop would return.  Slots are 32 bytes (one sector): three key words, the
// length (0 = empty) and the caller's id; open addressing, linear probing, load factor <= 0.5.
constexpr int TT_TOKTAB_MAXLEN = 24;
struct TokSlot { u64 k0, k1, k2; u32 len; int32_t id; };
static_assert(sizeof(TokSlot) == 32, "slot layout");
struct TokTable { const TokSlot* slots; u32 mask; u32 shift; };

TT_HD u32 toktab_hash(u64 k0, u64 k1, u64 k2, u32 len, u32 shift) {
    u64 h = (k0 + len) * 0x9E3779B97F4A7C15ull;
    h ^= (k1 + 0x632BE59BD9B4E019ull) * 0xC2B2AE3D27D4EB4Full;
    h ^= (k2 + 0x85157AF5ull) * 0x165667B19E3779F9ull;
    h ^= h >> 29;
    h *= 0xBF58476D1CE4E5B9ull;
    return (u32)(h >> shift);
}

// Key of a piece of 2..24 bytes: its bytes in three words, zero padded.
__device__ __forceinline__ void toktab_key(const u8* __restrict__ text, u32 a, u32 n, u64& k0, u64& k1, u64& k2) {
    // gather the piece's bytes with aligned 8-byte loads (only words that hold a piece byte)
    const uintptr_t addr = (uintptr_t)(text + a);
    const u64* w = reinterpret_cast<const u64*>(addr & ~(uintptr_t)7);
    const u32 sh = (u32)(addr & 7) * 8, last = (u32)(addr & 7) + n;     // bytes used in the window
    const u64 w0 = __ldg(w), w1 = last > 8 ? __ldg(w + 1) : 0, w2 = last > 16 ? __ldg(w + 2) : 0, w3 = last > 24 ? __ldg(w + 3) : 0;
    k0 = sh ? (w0 >> sh) | (w1 << (64 - sh)) : w0;
    k1 = sh ? (w1 >> sh) | (w2 << (64 - sh)) : w1;
    k2 = sh ? (w2 >> sh) | (w3 << (64 - sh)) : w2;
    if (n < 8) { k0 &= (1ull << (8 * n)) - 1; k1 = 0; k2 = 0; }
    else if (n < 16) { k1 &= (n == 8) ? 0 : ((1ull << (8 * (n - 8))) - 1); k2 = 0; }
    else if (n < 24) { k2 &= (n == 16) ? 0 : ((1ull << (8 * (n - 16))) - 1); }
}
// Probes from slot h on; lo / hi are the two halves of slot h, already loaded.
__device__ __forceinline__ bool toktab_finish(const TokTable& tab, u64 k0, u64 k1, u64 k2, u32 n, u32 h, uint4 lo, uint4 hi, int32_t& id) {
    for (u32 probe = 0; probe <= tab.mask; probe++) {           // bounded by the capacity
        if (hi.z == 0) return false;
        if (hi.z == n && (((u64)lo.y << 32) | lo.x) == k0 && (((u64)lo.w << 32) | lo.z) == k1 && (((u64)hi.y << 32) | hi.x) == k2) {
            id = (int32_t)hi.w;
            return true;
        }
        h = (h + 1) & tab.mask;
        const uint4* sp = reinterpret_cast<const uint4*>(tab.slots + h);
        lo = __ldg(sp); hi = __ldg(sp + 1);
    }
    return false;
}
// Looks a piece of 2..24 bytes up; returns true and the id on a hit.
__device__ __forceinline__ bool toktab_lookup(const TokTable& tab, const u8* __restrict__ text, u32 a, u32 n, int32_t& id) {
    u64 k0, k1, k2;
    toktab_key(text, a, n, k0, k1, k2);
    const u32 h = toktab_hash(k0, k1, k2, n, tab.shift);
    const uint4* sp = reinterpret_cast<const uint4*>(tab.slots + h);
    return toktab_finish(tab, k0, k1, k2, n, h, __ldg(sp), __ldg(sp + 1), id);
}

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

// ---- warp merge rounds with at most 32 tokens: one token per lane, no shared memory -----------------------
// t = token of position `lane`, r = rank of the pair (lane, lane + 1) or TT_RANK_INF, m = token count.
// Runs rounds to the fixpoint, stages the tokens (caller's ids) at stage[a ...] and returns their count.
__device__ __forceinline__ u32 warp_merge_reg_rounds(u32 t, u32 r, u32 m, u32 max_rounds, u32 a, const PairTable& tab,
                                                     const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage, int lane) {
    const u32 FULL = 0xFFFFFFFFu, lt = (1u << lane) - 1;
    for (u32 round = 0; round < max_rounds; round++) {
        const u32 mn = __reduce_min_sync(FULL, r);
        if (mn == TT_RANK_INF) break;
        // leftmost non-overlapping occurrences: inside a run of consecutive candidates, every other one
        const u32 c = __ballot_sync(FULL, r == mn);
        const u32 below = ~c & lt;
        const u32 dist = below ? (u32)(lane - (32 - __clz(below))) : (u32)lane;
        const u32 sel = __ballot_sync(FULL, ((c >> lane) & 1) && !(dist & 1));
        const bool me = (sel >> lane) & 1;
        const bool nxt = lane < 31 ? ((sel >> (lane + 1)) & 1) : false;
        const u32 nt = me ? 256u + mn : t;
        const u32 nr = (me || nxt) ? RK_STALE : r;
        // survivors move down: new lane j takes the j-th surviving old lane
        u32 src;
        if ((sel & (sel - 1)) == 0) {                   // one merge (the usual case): everything above it moves down by one
            src = (u32)lane + ((u32)lane > (u32)(__ffs(sel) - 1) ? 1u : 0u);
        } else {
            const u32 surv = ~(sel << 1) & (m >= 32 ? FULL : ((1u << m) - 1));
            src = __fns(surv, 0, lane + 1);
        }
        t = __shfl_sync(FULL, nt, src & 31);
        r = __shfl_sync(FULL, nr, src & 31);
        m -= __popc(sel);
        const u32 tn = __shfl_down_sync(FULL, t, 1);
        if ((u32)lane + 1 >= m) r = TT_RANK_INF;
        else if (r == RK_STALE) r = pair_probe(tab, t, tn);
    }
    if ((u32)lane < m) stage[a + lane] = ext_id[t];
    return m;
}

// A piece of up to 32 bytes.
__device__ __forceinline__ u32 warp_merge_reg(const u8* __restrict__ text, u32 a, u32 n, const PairTable& tab,
                                              const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage, int lane) {
    const u32 t = (u32)lane < n ? text[a + lane] : 0;
    const u32 tn = __shfl_down_sync(0xFFFFFFFFu, t, 1);
    const u32 r = ((u32)lane + 1 < n) ? __ldg(tab.bytepair + ((t << 8) | tn)) : TT_RANK_INF;
    return warp_merge_reg_rounds(t, r, n, n, a, tab, ext_id, stage, lane);
}

// ---- warp merge, 33..64 bytes: two tokens per lane, everything in registers ----------------------------------
// Position k lives in lane k % 32, register k / 32.  A round applies the occurrences of the minimum rank one
// after the other, leftmost first (a merge marks the pairs next to it stale, so an overlapping occurrence is
// no candidate any more: exactly the leftmost non-overlapping ones are taken); every step closes the gap
// with three shuffles per register pair instead of a trip through shared memory.  Then the stale pairs are
// probed together.  At 32 tokens the one-register rounds take over.
__device__ __forceinline__ u32 warp_merge_reg2(const u8* __restrict__ text, u32 a, u32 n, const PairTable& tab,
                                               const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage, int lane) {
    const u32 FULL = 0xFFFFFFFFu;
    u32 t0 = text[a + lane], t1 = 32u + lane < n ? text[a + 32 + lane] : 0u;
    u32 m = n;
    // pair (k, k + 1): right neighbour of position lane is (lane + 1, reg 0) or, for lane 31, (0, reg 1)
    u32 nx0 = __shfl_down_sync(FULL, t0, 1); { const u32 w = __shfl_sync(FULL, t1, 0); if (lane == 31) nx0 = w; }
    u32 nx1 = __shfl_down_sync(FULL, t1, 1);
    u32 r0 = (u32)lane + 1 < m ? __ldg(tab.bytepair + ((t0 << 8) | nx0)) : TT_RANK_INF;
    u32 r1 = 32u + lane + 1 < m ? __ldg(tab.bytepair + ((t1 << 8) | nx1)) : TT_RANK_INF;
    for (u32 round = 0; round < n && m > 32; round++) {
        const u32 mn = __reduce_min_sync(FULL, min(r0, r1));
        if (mn == TT_RANK_INF) break;
        for (u32 step = 0; step < 64; step++) {               // the occurrences of mn, leftmost first
            const u32 c0 = __ballot_sync(FULL, r0 == mn), c1 = __ballot_sync(FULL, r1 == mn);
            if (!(c0 | c1)) break;
            const u32 p = c0 ? (u32)__ffs(c0) - 1 : 32u + (u32)__ffs(c1) - 1;       // merge positions p, p + 1
            // new token at p, stale ranks at p - 1 and p, everything above p + 1 moves down by one
            const u32 d0 = __shfl_down_sync(FULL, t0, 1), d1 = __shfl_down_sync(FULL, t1, 1), w0 = __shfl_sync(FULL, t1, 0);
            const u32 e0 = __shfl_down_sync(FULL, r0, 1), e1 = __shfl_down_sync(FULL, r1, 1), x0 = __shfl_sync(FULL, r1, 0);
            const u32 k0 = lane, k1 = 32u + lane;
            const u32 up_t0 = lane == 31 ? w0 : d0, up_r0 = lane == 31 ? x0 : e0;        // old position k0 + 1
            const u32 up_t1 = lane == 31 ? 0u : d1, up_r1 = lane == 31 ? TT_RANK_INF : e1;  // old position k1 + 1
            t0 = k0 < p ? t0 : k0 == p ? 256u + mn : up_t0;
            r0 = k0 + 1 < p ? r0 : (k0 + 1 == p || k0 == p) ? RK_STALE : up_r0;
            t1 = k1 < p ? t1 : k1 == p ? 256u + mn : up_t1;
            r1 = k1 + 1 < p ? r1 : (k1 + 1 == p || k1 == p) ? RK_STALE : up_r1;
            m--;
            if (k0 + 1 >= m) r0 = TT_RANK_INF;                   // the last token has no pair
            if (k1 + 1 >= m) r1 = TT_RANK_INF;
        }
        nx0 = __shfl_down_sync(FULL, t0, 1); { const u32 w = __shfl_sync(FULL, t1, 0); if (lane == 31) nx0 = w; }
        nx1 = __shfl_down_sync(FULL, t1, 1);
        if (r0 == RK_STALE) r0 = pair_probe(tab, t0, nx0);
        if (r1 == RK_STALE) r1 = pair_probe(tab, t1, nx1);
    }
    if (m <= 32) return warp_merge_reg_rounds(t0, r0, m, m, a, tab, ext_id, stage, lane);
    if ((u32)lane < m) stage[a + lane] = ext_id[t0];
    if (32u + lane < m) stage[a + 32 + lane] = ext_id[t1];
    return m;
}

// ---- warp merge, 33..256 bytes: E tokens per lane in registers, compaction through shared memory ---------
// Position k lives in lane k % 32, register k / 32.  Each round the surviving (token, rank) pairs are
// written to their new positions in one of two shared-memory buffers (alternating, so one warp barrier
// per round suffices) and read back; ranks next to a merge are marked stale and probed again.
template <int E>
__device__ __forceinline__ u32 warp_merge_perm(u64* buf /* 2 * 32 * E entries of this warp */, const u8* __restrict__ text,
                                               u32 a, u32 n, const PairTable& tab, const int32_t* __restrict__ ext_id,
                                               int32_t* __restrict__ stage, int lane) {
    const u32 FULL = 0xFFFFFFFFu, lt = (1u << lane) - 1;
    u32 t[E], r[E];
    u32 m = n;
    __syncwarp();
#pragma unroll
    for (int j = 0; j < E; j++) {
        const u32 k = j * 32 + lane;
        t[j] = k < n ? text[a + k] : 0;
        buf[k] = t[j];
    }
    __syncwarp();
#pragma unroll
    for (int j = 0; j < E; j++) {
        const u32 k = j * 32 + lane;
        r[j] = (k + 1 < n) ? __ldg(tab.bytepair + ((t[j] << 8) | (u32)buf[k + 1])) : TT_RANK_INF;
    }
    int cur = 0;
    for (u32 round = 0; round < n; round++) {          // at most n - 1 merges
        u32 mn = r[0];
#pragma unroll
        for (int j = 1; j < E; j++) mn = min(mn, r[j]);
        mn = __reduce_min_sync(FULL, mn);
        if (mn == TT_RANK_INF) break;
        if (m <= 32) return warp_merge_reg_rounds(t[0], r[0], m, m, a, tab, ext_id, stage, lane);   // cheaper rounds from here on
        const int nch = (int)((m + 31) >> 5);
        u32 sel[E];
        u32 prev_ones = 0;                              // candidate run ending at the top of the previous word
#pragma unroll
        for (int j = 0; j < E; j++) {
            sel[j] = 0;
            if (j < nch) {
                const u32 c = __ballot_sync(FULL, r[j] == mn);
                const u32 below = ~c & lt;
                const u32 dist = below ? (u32)(lane - (32 - __clz(below))) : (u32)lane + prev_ones;
                sel[j] = __ballot_sync(FULL, ((c >> lane) & 1) && !(dist & 1));
                prev_ones = (c == FULL) ? prev_ones + 32 : (u32)__clz(~c);
            }
        }
        u64* nb = buf + (cur ^ 1) * (32 * E);
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
                    nb[np] = ((u64)((me || next_sel) ? RK_STALE : r[j]) << 32) | (me ? 256u + mn : t[j]);
                }
                removed += __popc(s);
            }
        }
        m -= removed;
        cur ^= 1;
        __syncwarp();
#pragma unroll
        for (int j = 0; j < E; j++) {
            const u32 k = j * 32 + lane;
            r[j] = TT_RANK_INF;
            if (k < m) {
                const u64 v = nb[k];
                t[j] = (u32)v;
                r[j] = (u32)(v >> 32);
                if (k + 1 >= m) r[j] = TT_RANK_INF;
                else if (r[j] == RK_STALE) r[j] = pair_probe(tab, t[j], (u32)nb[k + 1]);
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
// Two independent probes with both first-bucket loads in flight together.
__device__ __forceinline__ u32 pair_match_first(const PairTable& t, const uint4 lo, const uint4 hi, u64 key) {
    const u64 s0 = ((u64)lo.y << 32) | lo.x, s1 = ((u64)lo.w << 32) | lo.z, s2 = ((u64)hi.y << 32) | hi.x, s3 = ((u64)hi.w << 32) | hi.z;
    if ((s0 >> 20) == key) return (u32)(s0 & 0xFFFFFu);
    if ((s1 >> 20) == key) return (u32)(s1 & 0xFFFFFu);
    if ((s2 >> 20) == key) return (u32)(s2 & 0xFFFFFu);
    if ((s3 >> 20) == key) return (u32)(s3 & 0xFFFFFu);
    if (s3 == TT_SLOT_EMPTY) return TT_RANK_INF;
    return pair_probe(t, (u32)(key >> TT_ID_BITS), (u32)(key & (TT_MAX_INTERNAL - 1)));     // full bucket: walk the chain
}
__device__ __forceinline__ void pair_probe2(const PairTable& t, u32 a0, u32 b0, u32 a1, u32 b1, u32& r0, u32& r1) {
    const u64 key0 = ((u64)a0 << TT_ID_BITS) | b0, key1 = ((u64)a1 << TT_ID_BITS) | b1;
    const uint4* p0 = reinterpret_cast<const uint4*>(t.slots + 4 * (size_t)pair_bucket(key0, t.shift));
    const uint4* p1 = reinterpret_cast<const uint4*>(t.slots + 4 * (size_t)pair_bucket(key1, t.shift));
    const uint4 x0 = __ldg(p0), y0 = __ldg(p0 + 1), x1 = __ldg(p1), y1 = __ldg(p1 + 1);
    r0 = pair_match_first(t, x0, y0, key0);
    r1 = pair_match_first(t, x1, y1, key1);
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
        RK(k - 1) = __ldg(tab.bytepair + ((prev << 8) | t));
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
// arr[i] = token | (rank of the pair (i, i+1) << 32), in global scratch or shared memory.  One round:
// the minimum rank is found, every thread takes LK consecutive positions, decides which of its
// candidates are merged (the parity of a run of consecutive candidates is carried from thread to
// thread with one ballot-based scan; LK is even, so a slice that is all candidates leaves the parity
// unchanged), and the survivors are written to their new positions in place, chunk after chunk (every
// thread of a chunk has its positions in registers before anything is written, and writes never pass
// the read front).  Ranks next to a merge are marked stale and probed again in a second sweep, which
// also yields the next round's minimum.
constexpr int LK = 16;

__device__ __noinline__ u32 cta_merge_rounds(u64* arr, u32 m, const PairTable& tab, u32* s_scr /* >= 48 */, u32 stop_at, bool& finished) {
    const int tid = threadIdx.x, T = blockDim.x, lane = tid & 31, wid = tid >> 5, nw = T >> 5;
    finished = false;
    // minimum rank of the current array
    u32 lmin = TT_RANK_INF;
    for (u32 i = tid; i < m; i += T) lmin = min(lmin, (u32)(arr[i] >> 32));
    for (;;) {
        const u32 mn = cta_min_u32(lmin, s_scr);
        if (mn == TT_RANK_INF) { finished = true; return m; }
        if (m <= stop_at) return m;
        u32 carry_par = 0, out = 0;                        // parity of the candidate run before the chunk; survivors so far
        for (u32 base = 0; base < m; base += (u32)T * LK) {
            const u32 i0 = base + (u32)tid * LK;
            u32 tok[LK + 1], rk[LK + 1];
#pragma unroll
            for (int k = 0; k <= LK; k++) {
                const u32 i = i0 + k;
                const u64 v = i < m ? arr[i] : ~0ull;
                tok[k] = (u32)v; rk[k] = i < m ? (u32)(v >> 32) : TT_RANK_INF;
            }
            const u32 nval = i0 < m ? min((u32)LK, m - i0) : 0;
            u32 cand = 0;
#pragma unroll
            for (int k = 0; k <= LK; k++) cand |= (u32)(rk[k] == mn) << k;
            const u32 cand_in = cand & ((1u << LK) - 1);
            const bool all = cand_in == ((1u << LK) - 1);
            // parity of my trailing candidate run (if not all candidates)
            const u32 trail = __clz(~(cand_in << (32 - LK)));                 // consecutive candidates at the top of the slice
            const u32 my_par = trail & 1;
            // incoming parity: trailing parity of the nearest lower slice that is not all candidates
            const u32 allm = __ballot_sync(0xFFFFFFFFu, all), parm = __ballot_sync(0xFFFFFFFFu, my_par);
            const u32 lower = ~allm & ((1u << lane) - 1);
            __syncthreads();
            if (lane == 31) { const u32 na = ~allm; s_scr[wid] = na ? (2u | ((parm >> (31 - __clz(na))) & 1)) : 0u; }   // 0 = all lanes pass through
            __syncthreads();
            u32 in_par;
            if (lower) in_par = (parm >> (31 - __clz(lower))) & 1;
            else {
                in_par = carry_par;
                for (int w = wid - 1; w >= 0; w--) { const u32 e = s_scr[w]; if (e) { in_par = e & 1; break; } }
            }
            u32 next_carry = carry_par;
            for (int w = nw - 1; w >= 0; w--) { const u32 e = s_scr[w]; if (e) { next_carry = e & 1; break; } }
            // selection inside the slice (positions 0..LK; position LK only to know whether it is merged)
            u32 sel = 0, off = in_par;
#pragma unroll
            for (int k = 0; k <= LK; k++) {
                if ((cand >> k) & 1) { sel |= (u32)!(off & 1) << k; off++; } else off = 0;
            }
            const bool gone0 = in_par == 1;                                    // the element before the slice was merged with my first
            const u32 gone = ((sel << 1) | (u32)gone0) & ((1u << LK) - 1);
            const u32 valid = nval >= LK ? ((1u << LK) - 1) : ((1u << nval) - 1);
            const u32 surv = valid & ~gone;
            u32 tot;
            const u32 ex = cta_excl_sum_scan(__popc(surv), s_scr, &tot);         // all loads of the chunk are done: barrier inside
            u32 o = out + ex;
#pragma unroll
            for (int k = 0; k < LK; k++) {
                if ((surv >> k) & 1) {
                    const bool me = (sel >> k) & 1;
                    const bool nxt = me ? false : ((sel >> (k + 1)) & 1);
                    const u32 nt = me ? 256u + mn : tok[k];
                    const u32 nr = (me || nxt) ? RK_STALE : rk[k];
                    arr[o++] = ((u64)nr << 32) | nt;
                }
            }
            out += tot;
            carry_par = next_carry;
            __syncthreads();
        }
        m = out;
        __syncthreads();
        // probe the stale ranks again; collect the minimum for the next round
        lmin = TT_RANK_INF;
        for (u32 i = tid; i < m; i += T) {
            const u64 v = arr[i];
            u32 r = (u32)(v >> 32);
            if (i + 1 >= m) { r = TT_RANK_INF; arr[i] = ((u64)r << 32) | (u32)v; }
            else if (r == RK_STALE) { r = pair_probe(tab, (u32)v, (u32)arr[i + 1]); arr[i] = ((u64)r << 32) | (u32)v; }
            lmin = min(lmin, r);
        }
        __syncthreads();
    }
}

constexpr int LONG_SMEM_TOKENS = 4096;                  // long pieces move into shared memory below this many tokens

// Encodes one piece of n > TT_WARP_PIECE_MAX bytes with the whole CTA.  gbuf: n entries of global scratch.
__device__ u32 cta_merge_long(const u8* __restrict__ text, u32 a, u32 n, const PairTable& tab, const int32_t* __restrict__ ext_id,
                              int32_t* __restrict__ stage, u64* gbuf, u64* sbuf /* LONG_SMEM_TOKENS */, u32* s_scr) {
    const int tid = threadIdx.x, T = blockDim.x;
    u64* arr = n <= LONG_SMEM_TOKENS ? sbuf : gbuf;
    __syncthreads();
    for (u32 i = tid; i < n; i += T) {
        const u32 t0 = text[a + i];
        const u32 r = (i + 1 < n) ? __ldg(tab.bytepair + ((t0 << 8) | text[a + i + 1])) : TT_RANK_INF;
        arr[i] = ((u64)r << 32) | t0;
    }
    __syncthreads();
    bool finished;
    u32 m = cta_merge_rounds(arr, n, tab, s_scr, arr == gbuf ? LONG_SMEM_TOKENS : 0, finished);
    if (!finished && arr == gbuf) {
        __syncthreads();
        for (u32 i = tid; i < m; i += T) sbuf[i] = gbuf[i];
        __syncthreads();
        arr = sbuf;
        m = cta_merge_rounds(arr, m, tab, s_scr, 0, finished);
    }
    __syncthreads();
    for (u32 i = tid; i < m; i += T) stage[a + i] = ext_id[(u32)arr[i]];
    __syncthreads();
    return m;
}

// ---- pieces of one text tile -----------------------------------------------------------------------------
// The start flags of a tile (TT_TILE_CHUNKS u16 masks) become a list of in-tile piece offsets in shared
// memory; the end of the tile's last piece is the next start flag after the tile (or the text end).
constexpr int TILE_MAX_PIECES = TT_TILE_BYTES;

struct TilePieces {
    u16 off[TILE_MAX_PIECES];      // byte offset of each piece inside the tile (aligned frame)
    u32 n;                         // pieces that start in the tile
    u32 end;                       // end of the last piece, relative to the tile start (may lie far beyond the tile)
};

__device__ void tile_pieces(TilePieces& tp, const u16* __restrict__ startmask, const u32* __restrict__ tile_first,
                            long long nchunks, int ntiles, int tile, long long hi /* end of text, aligned frame */, u32* s_scr) {
    const int tid = threadIdx.x;
    const long long c0 = (long long)tile * TT_TILE_CHUNKS;
    u32 m = 0;
    if (tid < TT_TILE_CHUNKS && c0 + tid < nchunks) m = startmask[c0 + tid];
    if (tid == 0) {
        // the next start after the tile: the first start of the next tile that has one, else the text end
        u32 end = (u32)(hi - c0 * TT_CHUNK);
        for (int t = tile + 1; t < ntiles; t++) {
            const u32 f = tile_first[t];
            if (f != 0xFFFFFFFFu) { end = (u32)(t - tile) * TT_TILE_BYTES + f; break; }
        }
        tp.end = end;
    }
    u32 tot;
    u32 r = cta_excl_sum_scan(__popc(m), s_scr, &tot);
    while (m) { const int i = __ffs(m) - 1; m &= m - 1; tp.off[r++] = (u16)(tid * TT_CHUNK + i); }
    if (tid == 0) tp.n = tot;
    __syncthreads();
}

// ---- K4, first half: whole-piece lookups of a text tile; unsettled pieces go to global queues -----------------
// A thread per piece: one-byte pieces map directly, pieces of up to 24 bytes are looked up as whole
// vocabulary entries (two pieces per thread and step, their loads side by side).  What stays unsettled is
// appended to one of three queues in the workspace (one atomic reservation per tile and queue):
//   q_short  pieces of <= 32 bytes,  q_warp  pieces of 33..256 bytes,  q_long  longer pieces.
// Token totals of the settled pieces go to the per-tile and per-group counters.  This kernel holds no merge
// code, so it runs at full occupancy; k_merge then has every warp of the GPU drawing from the same queues.
// Without a token table (while the table itself is being built) every piece is queued.
struct PieceParams {
    const u8* base;            // aligned frame origin (text = base + shift)
    long long shift, hi;       // text occupies [shift, hi)
    long long nchunks;
    int ntiles;
    const u16* startmask;
    const u32* tile_first;     // offset of the first piece start inside every tile (~0: none)
    TTHeader* hdr;
    PairTable tab;
    TokTable toktab;
    const u32* litstart;       // literal pass: a piece that begins at such a bit is an added token whose id is staged, or null
    LongTable longtab;         // ignore_merges: entries longer than the whole-piece table holds (else slots == nullptr)
    const int32_t* ext_id;
    u32* piece_cnt;            // per piece: the id itself if the piece is one token found without merging (>= 0),
                               // else minus the number of tokens staged at the piece's text offset
    int32_t* stage;            // ids staged at the text offset of their piece
    u64* pairbuf;              // global scratch of the long-piece path, indexed like the text
    u32* tile_tok;             // in: zero; out: tokens per tile
    u32* grp_tok;              // in: zero; out: tokens per group of TT_GROUP_TILES tiles
    u64* q_short; u64* q_warp; // queue entries: text offset | index in tile << 32 | (bytes - 1) << 43
    uint4* q_long;             // (text offset, bytes, piece index, 0)
};

__device__ __forceinline__ u64 queue_entry(u32 a, u32 i, u32 n) { return (u64)a | ((u64)i << 32) | ((u64)(n - 1) << 43); }

constexpr int LOOKUP_THREADS = 256;
__global__ void __launch_bounds__(LOOKUP_THREADS, 6)
k_lookup(const PieceParams P) {
    __shared__ TilePieces tp;
    __shared__ u16 s_short[TILE_MAX_PIECES];                  // short misses from the front, long pieces from the back
    __shared__ u16 s_warp[TT_TILE_BYTES / (LANE_MAX + 1) + 2];
    __shared__ u32 s_ns, s_nw, s_nl, s_total, s_bs, s_bw, s_bl;
    __shared__ u32 sc[48];
    const int tid = threadIdx.x;
    cudaTriggerProgrammaticLaunchCompletion();               // the next kernel may be placed; it waits for this grid's memory itself
    if (P.toktab.slots != nullptr) grid_prefetch_l2(P.toktab.slots, ((size_t)P.toktab.mask + 1) * sizeof(TokSlot));
    cudaGridDependencySynchronize();                         // k_pretok's flags and counts are complete from here on
    const int status = P.hdr->status;                        // looked at after the first tile's flags are in: the loads overlap
    const u8* text = P.base + P.shift;
    for (int tile = blockIdx.x; tile < P.ntiles; tile += gridDim.x) {
        const long long c0 = (long long)tile * TT_TILE_CHUNKS;
        __syncthreads();
        if (tid == 0) { s_ns = 0; s_nw = 0; s_nl = 0; s_total = 0; }
        tile_pieces(tp, P.startmask, P.tile_first, P.nchunks, P.ntiles, tile, P.hi, sc);
        if (status != 0) return;                                  // nothing global has been written yet
        const u32 np = tp.n, p0 = (u32)tile * TT_TILE_BYTES;     // pieces are indexed per tile
        const long long t0 = c0 * TT_CHUNK - P.shift;             // text offset of the tile start
        u32 wsum = 0;
        // two pieces per thread and step, their loads issued side by side: first the bytes of both, then the
        // table slots of both (each lookup is a chain of two dependent loads)
        for (u32 ib = tid; ib < np; ib += 2 * LOOKUP_THREADS) {
            u32 a[2], n[2], h[2], kind[2];                        // kind: 0 none, 1 literal, 2 one byte, 3 table lookup, 4 other
            u64 k0[2], k1[2], k2[2];
            uint4 lo[2], hi[2];
#pragma unroll
            for (int j = 0; j < 2; j++) {
                const u32 i = ib + j * LOOKUP_THREADS;
                kind[j] = 0; a[j] = 0; n[j] = 0; k0[j] = 0; k1[j] = 0; k2[j] = 0;
                if (i < np) {
                    a[j] = (u32)(t0 + tp.off[i]);
                    n[j] = (i + 1 < np ? tp.off[i + 1] : tp.end) - tp.off[i];
                    const long long g = (long long)a[j] + P.shift;
                    if (P.litstart != nullptr && ((P.litstart[g >> 5] >> (g & 31)) & 1)) kind[j] = 1;
                    else if (n[j] == 1) { kind[j] = 2; k0[j] = text[a[j]]; }
                    else if (n[j] <= TT_TOKTAB_MAXLEN && P.toktab.slots != nullptr) { kind[j] = 3; toktab_key(text, a[j], n[j], k0[j], k1[j], k2[j]); }
                    else kind[j] = 4;
                }
            }
#pragma unroll
            for (int j = 0; j < 2; j++) {
                h[j] = 0; lo[j] = make_uint4(0, 0, 0, 0); hi[j] = lo[j];
                if (kind[j] == 3) {
                    h[j] = toktab_hash(k0[j], k1[j], k2[j], n[j], P.toktab.shift);
                    const uint4* sp = reinterpret_cast<const uint4*>(P.toktab.slots + h[j]);
                    lo[j] = __ldg(sp); hi[j] = __ldg(sp + 1);
                } else if (kind[j] == 2) lo[j].x = (u32)P.ext_id[(u32)k0[j]];
            }
#pragma unroll
            for (int j = 0; j < 2; j++) {
                const u32 i = ib + j * LOOKUP_THREADS;
                int32_t id;
                if (kind[j] == 0) continue;
                if (kind[j] == 1) { P.piece_cnt[p0 + i] = 0u - 1u; wsum++; }     // one staged id (written by the literal pass)
                else if (kind[j] == 2) { P.piece_cnt[p0 + i] = lo[j].x; wsum++; }
                else if (kind[j] == 3 && toktab_finish(P.toktab, k0[j], k1[j], k2[j], n[j], h[j], lo[j], hi[j], id)) {
                    P.piece_cnt[p0 + i] = (u32)id; wsum++;
                } else if (n[j] > TT_TOKTAB_MAXLEN && P.longtab.slots != nullptr && n[j] <= P.longtab.maxlen && longtab_lookup(P.longtab, text, a[j], n[j], id)) {
                    P.piece_cnt[p0 + i] = (u32)id; wsum++;
                } else if (n[j] > TT_WARP_PIECE_MAX) s_short[TILE_MAX_PIECES - 1 - atomicAdd(&s_nl, 1u)] = (u16)i;
                else if (n[j] > LANE_MAX) s_warp[atomicAdd(&s_nw, 1u)] = (u16)i;
                else s_short[atomicAdd(&s_ns, 1u)] = (u16)i;
            }
        }
        for (int o = 16; o; o >>= 1) wsum += __shfl_xor_sync(0xFFFFFFFFu, wsum, o);
        if ((tid & 31) == 0 && wsum) atomicAdd(&s_total, wsum);
        __syncthreads();
        const u32 ns = s_ns, nw = s_nw, nl = s_nl;
        if (tid == 0) {
            if (s_total) { atomicAdd(&P.tile_tok[tile], s_total); atomicAdd(&P.grp_tok[tile >> TT_GROUP_SHIFT], s_total); }
            if (ns) s_bs = atomicAdd(&P.hdr->nq_short, ns);
            if (nw) s_bw = atomicAdd(&P.hdr->nq_warp, nw);
            if (nl) s_bl = atomicAdd(&P.hdr->nq_long, nl);
        }
        if (ns | nw | nl) {                                       // block-uniform
            __syncthreads();
            for (u32 e = tid; e < ns + nw + nl; e += LOOKUP_THREADS) {
                const u32 i = e < ns ? s_short[e] : e < ns + nw ? s_warp[e - ns] : s_short[TILE_MAX_PIECES - 1 - (e - ns - nw)];
                const u32 a = (u32)(t0 + tp.off[i]);
                const u32 n = (i + 1 < np ? tp.off[i + 1] : tp.end) - tp.off[i];
                if (e < ns) P.q_short[s_bs + e] = queue_entry(a, i, n);
                else if (e < ns + nw) P.q_warp[s_bw + (e - ns)] = queue_entry(a, i, n);
                else P.q_long[s_bl + (e - ns - nw)] = make_uint4(a, n, p0 + i, 0u);
            }
        }
    }
}

// ---- K4, second half: the merges ------------------------------------------------------------------------------
// Long pieces (> 256 bytes) first, a CTA each.  Then every warp works on its own: it takes the pieces of
// 33..256 bytes one at a time (the longest chains, so they start first), then the pieces of <= 32 bytes --
// one at a time with the tokens in registers if the whole call has few of them (the shortest chain per piece:
// a request's latency is its longest chain), else 32 at a time, a thread per piece.  Tickets are global, so
// all warps of the GPU stay busy until the queues are empty; no barrier after the long pieces.
constexpr int MERGE_WARPS = 8;
constexpr int MERGE_THREADS = MERGE_WARPS * 32;
constexpr int WARP_SMEM_WORDS = 1024;                 // u64 per warp: two lane-path arrays of 32 x 32 u32, or the 2 x 256 merge buffers
static_assert(MERGE_WARPS * WARP_SMEM_WORDS >= LONG_SMEM_TOKENS, "the CTA's buffer must hold a long piece");
constexpr size_t MERGE_SMEM_BYTES = (size_t)MERGE_WARPS * WARP_SMEM_WORDS * sizeof(u64);   // dynamic shared memory of k_merge (64 KiB)
static_assert(WARP_SMEM_WORDS * sizeof(u64) >= 2 * LANE_SLOTS * LANE_MAX * sizeof(u32) && WARP_SMEM_WORDS >= 2 * TT_WARP_PIECE_MAX, "per-warp buffer");

__global__ void __launch_bounds__(MERGE_THREADS, 3)
k_merge(const PieceParams P) {
    extern __shared__ __align__(16) u64 s_buf[];              // MERGE_SMEM_BYTES
    __shared__ u32 sc[48];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    cudaTriggerProgrammaticLaunchCompletion();               // k_scatter may be placed; it waits for this grid's memory itself
    grid_prefetch_l2(P.tab.slots, ((size_t)P.tab.mask + 1) * 4 * sizeof(u64));
    grid_prefetch_l2(P.tab.bytepair, 65536 * sizeof(u32));
    cudaGridDependencySynchronize();                         // the queues are complete from here on
    if (P.hdr->status != 0) return;
    const u8* text = P.base + P.shift;
    const u32 ns = P.hdr->nq_short, nw = P.hdr->nq_warp, nl = P.hdr->nq_long;
    for (u32 e = blockIdx.x; e < nl; e += gridDim.x) {            // block-uniform
        const uint4 q = P.q_long[e];
        const u32 m = cta_merge_long(text, q.x, q.y, P.tab, P.ext_id, P.stage, P.pairbuf + q.x, s_buf, sc);
        if (tid == 0) {
            const u32 tile = q.z / TT_TILE_BYTES;
            P.piece_cnt[q.z] = 0u - m; atomicAdd(&P.tile_tok[tile], m); atomicAdd(&P.grp_tok[tile >> TT_GROUP_SHIFT], m);
        }
    }
    if (nl > blockIdx.x) __syncthreads();
    u64* wbuf = s_buf + wid * WARP_SMEM_WORDS;
    const u32 FULL = 0xFFFFFFFFu;
    for (;;) {                                                    // bounded by the queue length
        u32 e = 0;
        if (lane == 0) e = atomicAdd(&P.hdr->t_warp, 1u);
        e = __shfl_sync(FULL, e, 0);
        if (e >= nw) break;
        const u64 q = P.q_warp[e];
        const u32 a = (u32)q, i = (u32)(q >> 32) & 2047u, n = (u32)(q >> 43) + 1;
        const u32 m = n <= 64 ? warp_merge_reg2(text, a, n, P.tab, P.ext_id, P.stage, lane)
                              : warp_merge_perm<WCH>(wbuf, text, a, n, P.tab, P.ext_id, P.stage, lane);
        if (lane == 0) {
            const u32 tile = (u32)(((long long)a + P.shift) / TT_TILE_BYTES);
            P.piece_cnt[tile * TT_TILE_BYTES + i] = 0u - m; atomicAdd(&P.tile_tok[tile], m); atomicAdd(&P.grp_tok[tile >> TT_GROUP_SHIFT], m);
        }
    }
    if (ns <= 2u * MERGE_WARPS * gridDim.x) {                     // few: a warp per piece
        for (;;) {
            u32 e = 0;
            if (lane == 0) e = atomicAdd(&P.hdr->t_short, 1u);
            e = __shfl_sync(FULL, e, 0);
            if (e >= ns) break;
            const u64 q = P.q_short[e];
            const u32 a = (u32)q, i = (u32)(q >> 32) & 2047u, n = (u32)(q >> 43) + 1;
            const u32 m = warp_merge_reg(text, a, n, P.tab, P.ext_id, P.stage, lane);
            if (lane == 0) {
                const u32 tile = (u32)(((long long)a + P.shift) / TT_TILE_BYTES);
                P.piece_cnt[tile * TT_TILE_BYTES + i] = 0u - m; atomicAdd(&P.tile_tok[tile], m); atomicAdd(&P.grp_tok[tile >> TT_GROUP_SHIFT], m);
            }
        }
    } else {                                                      // bulk: 32 pieces per warp and step, a thread each
        u32* tok = reinterpret_cast<u32*>(wbuf);
        for (;;) {
            u32 e0 = 0;
            if (lane == 0) e0 = atomicAdd(&P.hdr->t_short, (u32)LANE_SLOTS);
            e0 = __shfl_sync(FULL, e0, 0);
            if (e0 >= ns) break;
            if (e0 + lane < ns) {
                const u64 q = P.q_short[e0 + lane];
                const u32 a = (u32)q, i = (u32)(q >> 32) & 2047u, n = (u32)(q >> 43) + 1;
                const u32 m = lane_merge(tok, tok + LANE_SLOTS * LANE_MAX, lane, text, a, n, P.tab, P.ext_id, P.stage);
                const u32 tile = (u32)(((long long)a + P.shift) / TT_TILE_BYTES);
                P.piece_cnt[tile * TT_TILE_BYTES + i] = 0u - m; atomicAdd(&P.tile_tok[tile], m); atomicAdd(&P.grp_tok[tile >> TT_GROUP_SHIFT], m);
            }
            __syncwarp();
        }
    }
}

// ---- K5: coalesced scatter of the staged ids, one text tile per CTA iteration ---------------------------------
// Also writes the token offset of every document that starts in the tile (batch calls).
struct ScatterParams {
    long long shift, hi, nchunks;
    int ntiles;
    const u16* startmask;
    const u32* tile_first;
    const u32* tile_tok;       // tokens per tile
    const u32* grp_tok;        // tokens per group of TT_GROUP_TILES tiles
    unsigned long long ids_cap;
    const u32* piece_cnt;
    const int32_t* stage;
    TTHeader* hdr;
    int32_t* ids_out;
    long long* count_out;
    int32_t* status_out;
    const u32* docmask;        // batch: bit per byte of document starts, else null
    const long long* doc_off;  // batch: n_docs + 1 offsets
    int n_docs;
    long long* ids_off_out;    // batch: n_docs + 1 token offsets
};

__global__ void __launch_bounds__(BPE_THREADS)
k_scatter(const ScatterParams P) {
    __shared__ TilePieces tp;
    __shared__ u32 sc[48];
    __shared__ u32 s_big[TILE_MAX_PIECES / 8][3];
    __shared__ u32 s_nbig;
    __shared__ unsigned long long s_sum[66];
    const int tid = threadIdx.x;
    cudaGridDependencySynchronize();                         // k_merge's (and with it k_lookup's) results are complete from here on
    // Each CTA takes a contiguous range of tiles.  Tokens before its first tile = the whole groups of tiles
    // before it plus the tiles of its own group before it; the grand total (all groups) gives the count and
    // the capacity check, which every CTA makes for itself.
    const int per = (P.ntiles + (int)gridDim.x - 1) / (int)gridDim.x;
    const int tile_lo = (int)blockIdx.x * per, tile_hi = min(P.ntiles, tile_lo + per);
    const int ngroups = (P.ntiles + TT_GROUP_TILES - 1) >> TT_GROUP_SHIFT, g_lo = tile_lo >> TT_GROUP_SHIFT;
    unsigned long long before = 0, total = 0;
    for (int g = tid; g < ngroups; g += BPE_THREADS) {
        const u32 x = P.grp_tok[g];
        total += x;
        if (g < g_lo) before += x;
    }
    for (int t = (g_lo << TT_GROUP_SHIFT) + tid; t < tile_lo; t += BPE_THREADS) before += P.tile_tok[t];
    cta_sum2_u64(before, total, s_sum);
    int status = P.hdr->status;
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
    u32 carry = (u32)before;
    for (int tile = tile_lo; tile < tile_hi; tile++) {
        const long long c0 = (long long)tile * TT_TILE_CHUNKS;
        __syncthreads();
        if (tid == 0) s_nbig = 0;
        tile_pieces(tp, P.startmask, P.tile_first, P.nchunks, P.ntiles, tile, P.hi, sc);
        const u32 np = tp.n, p0 = (u32)tile * TT_TILE_BYTES;
        const long long t0 = c0 * TT_CHUNK - P.shift;
        for (u32 b = 0; b < np; b += BPE_THREADS) {
            const u32 i = b + tid;
            const int32_t v = i < np ? (int32_t)P.piece_cnt[p0 + i] : 0;       // an id, or minus the staged count
            const u32 c = i < np ? (v >= 0 ? 1u : (u32)(-v)) : 0u;
            u32 tot;
            const u32 dst = carry + cta_excl_sum_scan(c, sc, &tot);
            if (i < np) {
                const u32 src = (u32)(t0 + tp.off[i]);
                if (v >= 0) P.ids_out[dst] = v;
                else if (c <= 8) { for (u32 k = 0; k < c; k++) P.ids_out[dst + k] = P.stage[src + k]; }
                else {
                    const u32 slot = atomicAdd(&s_nbig, 1u);
                    if (slot < TILE_MAX_PIECES / 8) { s_big[slot][0] = src; s_big[slot][1] = dst; s_big[slot][2] = c; }
                }
                if (P.docmask) {
                    const long long g = c0 * TT_CHUNK + tp.off[i];
                    if ((P.docmask[g >> 5] >> (g & 31)) & 1) {
                        // every document that starts at this byte (empty ones included) gets this token offset
                        const long long want = g - P.shift;
                        int lo = 0, hi2 = P.n_docs;
                        while (lo < hi2) { int mid = (lo + hi2) >> 1; if (P.doc_off[mid] < want) lo = mid + 1; else hi2 = mid; }
                        for (int d = lo; d <= P.n_docs && P.doc_off[d] == want; d++) P.ids_off_out[d] = dst;
                    }
                }
            }
            carry += tot;
            __syncthreads();
        }
        const u32 nbig = min(s_nbig, (u32)(TILE_MAX_PIECES / 8));
        for (u32 e = 0; e < nbig; e++) {
            const u32 src = s_big[e][0], d2 = s_big[e][1], cc = s_big[e][2];
            for (u32 k = tid; k < cc; k += BPE_THREADS) P.ids_out[d2 + k] = P.stage[src + k];
        }
    }
}

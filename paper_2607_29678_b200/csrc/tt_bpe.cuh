// Steps K4 and K5: byte-level BPE per piece, token counts and scatter of the IDs.
//
// Paper Sec. 4.2: every piece is encoded independently; merge ranks and vocabulary entries live in
// GPU hash tables; a round's minimum rank identifies one pair value, merging all its leftmost
// non-overlapping occurrences equals iterated single merges, and only pairs next to a completed
// merge need to be probed again.  Work is dispatched by piece length and difficulty:
//   * a thread per piece looks the whole piece up as a vocabulary entry (one 32-byte probe);
//   * pieces that are not a single entry are merged by a warp (<= 32 bytes: tokens in registers,
//     candidates as ballot masks; <= 256 bytes: several tokens per lane, compaction through shared memory);
//   * longer pieces are merged by a whole CTA with its state in global scratch (k_bpe_long).
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
    u32 mask;             // number of buckets - 1 (power of two)
    u32 shift;            // 64 - log2(number of buckets)
};
TT_HD u32 pair_bucket(u64 key, u32 shift) { return (u32)((key * 0x9E3779B97F4A7C15ull) >> shift); }

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

// Looks a piece of 2..24 bytes up; returns true and the id on a hit.
__device__ __forceinline__ bool toktab_lookup(const TokTable& tab, const u8* __restrict__ text, u32 a, u32 n, int32_t& id) {
    // gather the piece's bytes with aligned 8-byte loads (only words that hold a piece byte)
    const uintptr_t addr = (uintptr_t)(text + a);
    const u64* w = reinterpret_cast<const u64*>(addr & ~(uintptr_t)7);
    const u32 sh = (u32)(addr & 7) * 8, last = (u32)(addr & 7) + n;     // bytes used in the window
    const u64 w0 = __ldg(w), w1 = last > 8 ? __ldg(w + 1) : 0, w2 = last > 16 ? __ldg(w + 2) : 0, w3 = last > 24 ? __ldg(w + 3) : 0;
    u64 k0 = sh ? (w0 >> sh) | (w1 << (64 - sh)) : w0;
    u64 k1 = sh ? (w1 >> sh) | (w2 << (64 - sh)) : w1;
    u64 k2 = sh ? (w2 >> sh) | (w3 << (64 - sh)) : w2;
    if (n < 8) { k0 &= (1ull << (8 * n)) - 1; k1 = 0; k2 = 0; }
    else if (n < 16) { k1 &= (n == 8) ? 0 : ((1ull << (8 * (n - 8))) - 1); k2 = 0; }
    else if (n < 24) { k2 &= (n == 16) ? 0 : ((1ull << (8 * (n - 16))) - 1); }
    u32 h = toktab_hash(k0, k1, k2, n, tab.shift);
    for (u32 probe = 0; probe <= tab.mask; probe++) {           // bounded by the capacity
        const uint4* sp = reinterpret_cast<const uint4*>(tab.slots + h);
        const uint4 lo = __ldg(sp), hi = __ldg(sp + 1);
        if (hi.z == 0) return false;
        if (hi.z == n && (((u64)lo.y << 32) | lo.x) == k0 && (((u64)lo.w << 32) | lo.z) == k1 && (((u64)hi.y << 32) | hi.x) == k2) {
            id = (int32_t)hi.w;
            return true;
        }
        h = (h + 1) & tab.mask;
    }
    return false;
}

constexpr u32 RK_STALE = 0xFFFFFFFEu;                 // rank must be probed again
constexpr int BPE_WARPS = 8;                          // warps per CTA of the piece kernels
constexpr int BPE_THREADS = BPE_WARPS * 32;           // = pieces per CTA iteration
constexpr int WCH = TT_WARP_PIECE_MAX / 32;           // 32-token chunks per piece

// ---- warp merge, up to 32 bytes: one token per lane, no shared memory ------------------------------------
// Returns the token count; the tokens (caller's ids) are staged at stage[a ...].
__device__ __forceinline__ u32 warp_merge_reg(const u8* __restrict__ text, u32 a, u32 n, const PairTable& tab,
                                              const int32_t* __restrict__ ext_id, int32_t* __restrict__ stage, int lane) {
    const u32 FULL = 0xFFFFFFFFu, lt = (1u << lane) - 1;
    u32 t = (u32)lane < n ? text[a + lane] : 0;
    u32 m = n;
    u32 tn = __shfl_down_sync(FULL, t, 1);
    u32 r = ((u32)lane + 1 < m) ? pair_probe(tab, t, tn) : TT_RANK_INF;
    for (u32 round = 0; round < n; round++) {          // at most n - 1 merges
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
        const u32 surv = ~(sel << 1) & (m >= 32 ? FULL : ((1u << m) - 1));
        const u32 src = __fns(surv, 0, lane + 1);
        t = __shfl_sync(FULL, nt, src & 31);
        r = __shfl_sync(FULL, nr, src & 31);
        m -= __popc(sel);
        tn = __shfl_down_sync(FULL, t, 1);
        if ((u32)lane + 1 >= m) r = TT_RANK_INF;
        else if (r == RK_STALE) r = pair_probe(tab, t, tn);
    }
    if ((u32)lane < m) stage[a + lane] = ext_id[t];
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
        r[j] = (k + 1 < n) ? pair_probe(tab, t[j], (u32)buf[k + 1]) : TT_RANK_INF;
    }
    int cur = 0;
    for (u32 round = 0; round < n; round++) {          // at most n - 1 merges
        u32 mn = r[0];
#pragma unroll
        for (int j = 1; j < E; j++) mn = min(mn, r[j]);
        mn = __reduce_min_sync(FULL, mn);
        if (mn == TT_RANK_INF) break;
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

// ---- CTA-wide scans -----------------------------------------------------------------------------------
__device__ __forceinline__ int cta_incl_max_scan(int v, int* scratch /* >= 33 */, int carry) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xFFFFFFFFu, v, o); if (lane >= o) v = max(v, t); }
    __syncthreads();
    if (lane == 31) scratch[wid] = v;
    __syncthreads();
    if (wid == 0) {
        int s = lane < nw ? scratch[lane] : INT_MIN;
        for (int o = 1; o < 32; o <<= 1) { int t = __shfl_up_sync(0xFFFFFFFFu, s, o); if (lane >= o) s = max(s, t); }
        if (lane < nw) scratch[lane] = s;
    }
    __syncthreads();
    int before = wid ? scratch[wid - 1] : INT_MIN;
    return max(max(v, before), carry);
}
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

// ---- K4, pieces of a block of BPE_THREADS consecutive pieces ---------------------------------------------
// Phase 1: a thread per piece (one-byte pieces map directly, pieces of up to 24 bytes are looked up as
// whole vocabulary entries).  Phase 2: the CTA's warps merge the pieces phase 1 could not settle.
// Phase 3: the token total of the block; the last CTA to finish turns the block totals into their
// exclusive prefix (K5's scan) and checks the output capacity.  Pieces longer than
// TT_WARP_PIECE_MAX were encoded before this kernel (k_bpe_long); only their counts are read here.
// Without a token table (while the table itself is being built) every piece takes the merge path.
__global__ void __launch_bounds__(BPE_THREADS)
k_bpe_pieces(const u8* __restrict__ text, const u32* __restrict__ piece_off, TTHeader* hdr, const PairTable tab,
             const TokTable toktab, const int32_t* __restrict__ ext_id, u32* __restrict__ piece_cnt,
             int32_t* __restrict__ stage, u32* __restrict__ blk_cnt, unsigned long long ids_cap) {
    __shared__ u64 s_buf[BPE_WARPS][2 * TT_WARP_PIECE_MAX];     // two (token, rank) buffers per warp
    __shared__ u32 s_miss[BPE_THREADS];
    __shared__ u32 s_nmiss, s_total, s_islast;
    __shared__ u32 sc[40];
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
    const bool dead = hdr->status != 0;
    const u32 n_pieces = dead ? 0 : hdr->n_pieces;
    const u32 n_blocks = (n_pieces + BPE_THREADS - 1) / BPE_THREADS;
    for (u32 pb = blockIdx.x; pb < n_blocks; pb += gridDim.x) {
        __syncthreads();
        if (tid == 0) { s_nmiss = 0; s_total = 0; }
        __syncthreads();
        const u32 p = pb * BPE_THREADS + tid;
        u32 cnt = 0;
        if (p < n_pieces) {
            const u32 a = piece_off[p], n = piece_off[p + 1] - a;
            int32_t id;
            if (n == 1) { stage[a] = ext_id[text[a]]; cnt = 1; }
            else if (n > TT_WARP_PIECE_MAX) cnt = piece_cnt[p];
            else if (n <= TT_TOKTAB_MAXLEN && toktab.slots != nullptr && toktab_lookup(toktab, text, a, n, id)) { stage[a] = id; cnt = 1; }
            else s_miss[atomicAdd(&s_nmiss, 1u)] = p;
            if (cnt && n <= TT_WARP_PIECE_MAX) piece_cnt[p] = cnt;
        }
        u32 wsum = cnt;
        for (int o = 16; o; o >>= 1) wsum += __shfl_xor_sync(0xFFFFFFFFu, wsum, o);
        __syncthreads();
        const u32 nmiss = s_nmiss;
        u32 msum = 0;
        for (u32 e = wid; e < nmiss; e += BPE_WARPS) {
            const u32 q = s_miss[e];
            const u32 a = piece_off[q], n = piece_off[q + 1] - a;
            const u32 m = n <= 32 ? warp_merge_reg(text, a, n, tab, ext_id, stage, lane)
                        : n <= 64 ? warp_merge_perm<2>(s_buf[wid], text, a, n, tab, ext_id, stage, lane)
                                  : warp_merge_perm<WCH>(s_buf[wid], text, a, n, tab, ext_id, stage, lane);
            if (lane == 0) piece_cnt[q] = m;
            msum += m;
        }
        if (lane == 0) atomicAdd(&s_total, wsum + msum);
        __syncthreads();
        if (tid == 0) blk_cnt[pb] = s_total;
    }
    // the last CTA to finish: exclusive prefix of the block totals, total token count, capacity check
    __threadfence();
    __syncthreads();
    if (tid == 0) s_islast = (atomicAdd(&hdr->count_done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!s_islast) return;
    __threadfence();
    unsigned long long carry = 0;
    for (u32 b0 = 0; b0 < n_blocks; b0 += BPE_THREADS) {
        const u32 i = b0 + tid;
        u32 x = i < n_blocks ? blk_cnt[i] : 0, t2;
        const u32 ex = cta_excl_sum_scan(x, sc, &t2);
        if (i < n_blocks) blk_cnt[i] = (u32)carry + ex;
        carry += t2;
        __syncthreads();
    }
    if (tid == 0) {
        hdr->n_tokens = carry;
        if (!dead && carry > ids_cap) atomicMax(&hdr->status, 5 /* TT_ERR_CAPACITY */);
    }
}

// ---- K4, CTA per long piece (long whitespace / punctuation runs and other pieces > 256 bytes) -----
constexpr int LONG_THREADS = 1024;
constexpr u32 TOK_NEW = 0x80000000u;                  // token produced in the current round

__global__ void __launch_bounds__(LONG_THREADS)
k_bpe_long(const u8* __restrict__ text, const u32* __restrict__ piece_off, TTHeader* hdr, const PairTable tab,
           const int32_t* __restrict__ ext_id, u32* __restrict__ piece_cnt, int32_t* __restrict__ stage,
           u32* __restrict__ rank_buf, const u32* __restrict__ long_list) {
    __shared__ u32 s_u[40];
    __shared__ int s_i[40];
    __shared__ u32 s_sel[LONG_THREADS];
    __shared__ u32 s_item, s_min;
    if (hdr->status != 0) return;
    const u32 n_long = hdr->n_long;
    const int tid = threadIdx.x;
    for (;;) {
        __syncthreads();
        if (tid == 0) s_item = atomicAdd(&hdr->long_next, 1u);
        __syncthreads();
        const u32 item = s_item;
        if (item >= n_long) break;
        const u32 p = long_list[item];
        const u32 a = piece_off[p], n = piece_off[p + 1] - a;
        u32* tok = reinterpret_cast<u32*>(stage) + a;
        u32* rk = rank_buf + a;
        for (u32 i = tid; i < n; i += LONG_THREADS) tok[i] = text[a + i];
        __syncthreads();
        for (u32 i = tid; i < n; i += LONG_THREADS) rk[i] = (i + 1 < n) ? pair_probe(tab, tok[i], tok[i + 1]) : TT_RANK_INF;
        u32 m = n;
        for (u32 round = 0; round < n; round++) {
            __syncthreads();
            // pass 1: minimum rank present
            u32 mn = TT_RANK_INF;
            for (u32 i = tid; i < m; i += LONG_THREADS) mn = min(mn, rk[i]);
            mn = __reduce_min_sync(0xFFFFFFFFu, mn);
            if (tid == 0) s_min = TT_RANK_INF;
            __syncthreads();
            if ((tid & 31) == 0) atomicMin(&s_min, mn);
            __syncthreads();
            mn = s_min;
            if (mn == TT_RANK_INF) break;
            // pass 2: select and compact, chunk by chunk in order (writes never pass the read front)
            int carry_z = -1;            // nearest non-candidate position so far
            u32 carry_removed = 0, carry_lastsel = 0;
            for (u32 b = 0; b < m; b += LONG_THREADS) {
                const u32 i = b + tid;
                const bool in = i < m;
                const u32 t = in ? (tok[i] & ~TOK_NEW) : 0;
                const u32 r = in ? rk[i] : TT_RANK_INF;
                const bool cand = in && r == mn;
                const int z = cta_incl_max_scan(cand ? -1 : (int)i, s_i, carry_z);
                const bool sel = cand && !(((int)i - z - 1) & 1);
                s_sel[tid] = sel;
                u32 tot;
                const u32 ex = cta_excl_sum_scan(sel ? 1u : 0u, s_u, &tot);     // contains __syncthreads: s_sel visible
                const bool gone = tid ? s_sel[tid - 1] : carry_lastsel;
                if (in && !gone) {
                    const u32 np = i - carry_removed - ex;
                    tok[np] = sel ? ((256u + mn) | TOK_NEW) : t;
                    rk[np] = r;
                }
                // carries for the next chunk (identical in every thread)
                const u32 last = min(m - b, (u32)LONG_THREADS) - 1;
                __syncthreads();
                if (tid == (int)last) { s_i[34] = z; s_u[34] = sel; }
                __syncthreads();
                carry_z = s_i[34]; carry_lastsel = s_u[34];
                carry_removed += tot;
            }
            m -= carry_removed;
            __syncthreads();
            // pass 3: probe again the pairs that touch a new token
            for (u32 i = tid; i < m; i += LONG_THREADS) {
                const u32 x = tok[i], y = (i + 1 < m) ? tok[i + 1] : 0;
                if ((x | y) & TOK_NEW) rk[i] = (i + 1 < m) ? pair_probe(tab, x & ~TOK_NEW, y & ~TOK_NEW) : TT_RANK_INF;
            }
        }
        __syncthreads();
        for (u32 i = tid; i < m; i += LONG_THREADS) stage[a + i] = ext_id[tok[i] & ~TOK_NEW];
        if (tid == 0) piece_cnt[p] = m;
    }
}

// ---- K5: token offsets per piece and coalesced scatter of the staged ids ----------------------------------
// One CTA per block of BPE_THREADS pieces (the same partition as k_bpe_pieces, whose last CTA left the
// exclusive prefix of the block totals in blk_base).
__global__ void __launch_bounds__(BPE_THREADS)
k_scatter(const u32* __restrict__ piece_off, const u32* __restrict__ piece_cnt, const u32* __restrict__ blk_base,
          const int32_t* __restrict__ stage, TTHeader* hdr, u32* __restrict__ tok_off, int32_t* __restrict__ ids_out,
          long long* __restrict__ count_out, int32_t* __restrict__ status_out) {
    __shared__ u32 sc[40];
    __shared__ u32 s_big[BPE_THREADS][3];
    __shared__ u32 s_nbig;
    const int status = hdr->status;
    const u32 n_pieces = hdr->n_pieces;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (status_out) *status_out = status;
        if (count_out) *count_out = status ? 0 : (long long)hdr->n_tokens;
        if (status || n_pieces == 0) tok_off[0] = 0;
    }
    if (status != 0) return;
    const u32 n_blocks = (n_pieces + BPE_THREADS - 1) / BPE_THREADS;
    for (u32 pb = blockIdx.x; pb < n_blocks; pb += gridDim.x) {
        __syncthreads();
        if (threadIdx.x == 0) s_nbig = 0;
        const u32 p = pb * BPE_THREADS + threadIdx.x;
        const u32 c = p < n_pieces ? piece_cnt[p] : 0;
        u32 tot;
        const u32 dst = blk_base[pb] + cta_excl_sum_scan(c, sc, &tot);
        if (p < n_pieces) {
            tok_off[p] = dst;
            if (p == n_pieces - 1) tok_off[n_pieces] = dst + c;
            const u32 src = piece_off[p];
            if (c <= 8) {
                for (u32 k = 0; k < c; k++) ids_out[dst + k] = stage[src + k];
            } else {
                const u32 slot = atomicAdd(&s_nbig, 1u);
                s_big[slot][0] = src; s_big[slot][1] = dst; s_big[slot][2] = c;
            }
        }
        __syncthreads();
        const u32 nbig = s_nbig;
        for (u32 e = 0; e < nbig; e++) {
            const u32 src = s_big[e][0], d2 = s_big[e][1], cc = s_big[e][2];
            for (u32 k = threadIdx.x; k < cc; k += BPE_THREADS) ids_out[d2 + k] = stage[src + k];
        }
    }
}

// ---- batch: token offset of every document ----------------------------------------------------------
__global__ void k_doc_offsets(const long long* __restrict__ doc_off, int n_docs, const u32* __restrict__ piece_off,
                              const u32* __restrict__ tok_off, const TTHeader* hdr, long long* __restrict__ ids_off_out) {
    const int d = blockIdx.x * blockDim.x + threadIdx.x;
    if (d > n_docs) return;
    if (hdr->status != 0) { ids_off_out[d] = 0; return; }
    const u32 n_pieces = hdr->n_pieces;
    const long long want = doc_off[d];
    u32 lo = 0, hi = n_pieces;                  // first piece whose offset is >= want
    while (lo < hi) { u32 mid = (lo + hi) >> 1; if ((long long)piece_off[mid] < want) lo = mid + 1; else hi = mid; }
    ids_off_out[d] = tok_off[lo];
}

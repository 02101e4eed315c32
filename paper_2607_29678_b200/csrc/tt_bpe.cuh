// Steps K4 and K5: byte-level BPE per piece, token-count scan and scatter of the IDs.
//
// Paper Sec. 4.2: every piece is encoded independently; merge ranks live in a GPU hash table; a
// round's minimum rank identifies one pair value, merging all its leftmost non-overlapping
// occurrences equals iterated single merges, and only pairs next to a completed merge need to be
// probed again.  Work is dispatched by piece length: a warp per piece up to TT_WARP_PIECE_MAX
// bytes (state in shared memory, candidates as ballot masks), a CTA per longer piece (state in
// global scratch).  Token ids used inside the kernels are "internal": byte b -> b, result of the
// merge of rank r -> 256 + r; the caller's ids are looked up when the tokens are staged.
#pragma once
#include "tt_common.cuh"

struct PairTable {
    const u64* slots;     // open addressing, linear probing; slot = (left << 38) | (right << 20) | rank
    u32 mask;             // capacity - 1 (capacity is a power of two, load factor <= 0.5)
    u32 shift;            // 64 - log2(capacity)
};

__device__ __forceinline__ u32 pair_probe(const PairTable& t, u32 a, u32 b) {
    const u64 key = ((u64)a << TT_ID_BITS) | b;
    u32 h = (u32)((key * 0x9E3779B97F4A7C15ull) >> t.shift);
    for (u32 n = 0; n <= t.mask; n++) {               // bounded by the table capacity
        const u64 s = __ldg(t.slots + h);
        if (s == TT_SLOT_EMPTY) return TT_RANK_INF;
        if ((s >> 20) == key) return (u32)(s & 0xFFFFFu);
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

// K4, thread per piece: one-byte pieces map directly; pieces of up to 24 bytes are looked up as whole
// vocabulary entries; everything else (and every miss) goes to the miss list for the merge kernels.
__global__ void __launch_bounds__(256)
k_bpe_lookup(const u8* __restrict__ text, const u32* __restrict__ piece_off, TTHeader* hdr, const TokTable tab,
             const int32_t* __restrict__ ext_id, u32* __restrict__ piece_cnt, int32_t* __restrict__ stage,
             u32* __restrict__ miss_list) {
    if (hdr->status != 0) return;
    const u32 n_pieces = hdr->n_pieces;
    const u32 lane = threadIdx.x & 31;
    const u32 stride = gridDim.x * blockDim.x;
    const u32 rounds = (n_pieces + stride - 1) / stride;
    u32 p = blockIdx.x * blockDim.x + threadIdx.x;
    for (u32 it = 0; it < rounds; it++, p += stride) {
        bool miss = false;
        if (p < n_pieces) {
            const u32 a = piece_off[p], n = piece_off[p + 1] - a;
            if (n == 1) {
                stage[a] = ext_id[text[a]]; piece_cnt[p] = 1;
            } else if (n > TT_TOKTAB_MAXLEN || tab.slots == nullptr) {
                miss = true;
            } else {
                // gather the piece's bytes with aligned 8-byte loads (only words that hold a piece byte)
                const uintptr_t addr = (uintptr_t)(text + a);
                const u64* w = reinterpret_cast<const u64*>(addr & ~(uintptr_t)7);
                const u32 sh = (u32)(addr & 7) * 8, last = (u32)(addr & 7) + n;     // bytes used in the window
                const u64 w0 = __ldg(w), w1 = last > 8 ? __ldg(w + 1) : 0, w2 = last > 16 ? __ldg(w + 2) : 0,
                          w3 = last > 24 ? __ldg(w + 3) : 0;
                u64 k0 = sh ? (w0 >> sh) | (w1 << (64 - sh)) : w0;
                u64 k1 = sh ? (w1 >> sh) | (w2 << (64 - sh)) : w1;
                u64 k2 = sh ? (w2 >> sh) | (w3 << (64 - sh)) : w2;
                if (n < 8) { k0 &= (1ull << (8 * n)) - 1; k1 = 0; k2 = 0; }
                else if (n < 16) { k1 &= (n == 8) ? 0 : ((1ull << (8 * (n - 8))) - 1); k2 = 0; }
                else if (n < 24) { k2 &= (n == 16) ? 0 : ((1ull << (8 * (n - 16))) - 1); }
                u32 h = toktab_hash(k0, k1, k2, n, tab.shift);
                miss = true;
                for (u32 probe = 0; probe <= tab.mask; probe++) {           // bounded by the capacity
                    const uint4* sp = reinterpret_cast<const uint4*>(tab.slots + h);
                    const uint4 lo = __ldg(sp), hi = __ldg(sp + 1);
                    const u32 slen = hi.z;
                    if (slen == 0) break;
                    if (slen == n && (((u64)lo.y << 32) | lo.x) == k0 && (((u64)lo.w << 32) | lo.z) == k1 &&
                        (((u64)hi.y << 32) | hi.x) == k2) {
                        stage[a] = (int32_t)hi.w; piece_cnt[p] = 1; miss = false; break;
                    }
                    h = (h + 1) & tab.mask;
                }
            }
        }
        const u32 mm = __ballot_sync(0xFFFFFFFFu, miss);
        if (mm) {
            u32 base = 0;
            if (lane == 0) base = atomicAdd(&hdr->n_miss, (u32)__popc(mm));
            base = __shfl_sync(0xFFFFFFFFu, base, 0);
            if (miss) miss_list[base + __popc(mm & ((1u << lane) - 1))] = p;
        }
    }
}

constexpr u32 RK_STALE = 0xFFFFFFFEu;                 // rank must be probed again
constexpr int BPE_WARPS = 8;                          // warps per CTA of the warp-per-piece kernel
constexpr int WCH = TT_WARP_PIECE_MAX / 32;           // 32-token chunks per piece

// ---- K4, warp per piece ---------------------------------------------------------------------------
__global__ void __launch_bounds__(BPE_WARPS * 32)
k_bpe_warp(const u8* __restrict__ text, const u32* __restrict__ piece_off, TTHeader* hdr, const PairTable tab,
           const int32_t* __restrict__ ext_id, u32* __restrict__ piece_cnt, int32_t* __restrict__ stage,
           u32* __restrict__ long_list, const u32* __restrict__ miss_list) {
    __shared__ u32 s_tok[BPE_WARPS][TT_WARP_PIECE_MAX];
    __shared__ u32 s_rk[BPE_WARPS][TT_WARP_PIECE_MAX];
    if (hdr->status != 0) return;
    // with a miss list: the pieces the lookup kernel could not settle; without: every piece
    const u32 n_items = miss_list ? hdr->n_miss : hdr->n_pieces;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const u32 lt = (1u << lane) - 1;
    u32* tok = s_tok[wid];
    u32* rk = s_rk[wid];
    const u32 nwarps = gridDim.x * BPE_WARPS;
    for (u32 item = blockIdx.x * BPE_WARPS + wid; item < n_items; item += nwarps) {
        const u32 p = miss_list ? miss_list[item] : item;
        const u32 a = piece_off[p], n = piece_off[p + 1] - a;
        if (n > TT_WARP_PIECE_MAX) {
            if (lane == 0) long_list[atomicAdd(&hdr->n_long, 1u)] = p;
            continue;
        }
        if (n == 1) {
            if (lane == 0) { stage[a] = ext_id[text[a]]; piece_cnt[p] = 1; }
            continue;
        }
        __syncwarp();
        for (u32 k = lane; k < n; k += 32) tok[k] = text[a + k];
        __syncwarp();
        for (u32 k = lane; k < n; k += 32) rk[k] = (k + 1 < n) ? pair_probe(tab, tok[k], tok[k + 1]) : TT_RANK_INF;
        u32 m = n;
        for (u32 round = 0; round < n; round++) {      // at most n - 1 merges
            __syncwarp();
            const int nch = (int)((m + 31) >> 5);
            u32 t[WCH], r[WCH];
            u32 mn = TT_RANK_INF;
#pragma unroll
            for (int j = 0; j < WCH; j++) {
                if (j < nch) {
                    const u32 k = j * 32 + lane;
                    t[j] = k < m ? tok[k] : 0;
                    r[j] = k < m ? rk[k] : TT_RANK_INF;
                    mn = min(mn, r[j]);
                }
            }
            mn = __reduce_min_sync(0xFFFFFFFFu, mn);
            if (mn == TT_RANK_INF) break;
            // candidates, then leftmost non-overlapping selection: inside a maximal run of
            // consecutive candidates take the positions at even distance from the run start
            u32 sel[WCH];
            u32 prev_ones = 0;                          // length of the candidate run that ends at the previous chunk's top
#pragma unroll
            for (int j = 0; j < WCH; j++) {
                if (j < nch) {
                    const u32 c = __ballot_sync(0xFFFFFFFFu, r[j] == mn);
                    const u32 below = ~c & lt;
                    const u32 dist = below ? (u32)(lane - (32 - __clz(below))) : (u32)lane + prev_ones;
                    sel[j] = __ballot_sync(0xFFFFFFFFu, ((c >> lane) & 1) && !(dist & 1));
                    prev_ones = (c == 0xFFFFFFFFu) ? prev_ones + 32 : (u32)__clz(~c);
                }
            }
            __syncwarp();
            // compaction in place: every lane has read its elements; survivors move down
            u32 removed = 0;
#pragma unroll
            for (int j = 0; j < WCH; j++) {
                if (j < nch) {
                    const u32 k = j * 32 + lane;
                    const u32 s = sel[j];
                    const bool me = (s >> lane) & 1;
                    const bool gone = lane ? ((s >> (lane - 1)) & 1) : (j ? (sel[j - 1] >> 31) & 1 : 0);
                    const bool next_sel = lane < 31 ? ((s >> (lane + 1)) & 1) : ((j + 1 < nch) ? (sel[j + 1] & 1) : 0);
                    if (k < m && !gone) {
                        const u32 np = k - removed - __popc(s & lt);
                        tok[np] = me ? 256u + mn : t[j];
                        rk[np] = (me || next_sel) ? RK_STALE : r[j];
                    }
                    removed += __popc(s);
                }
            }
            m -= removed;
            __syncwarp();
            for (u32 k = lane; k < m; k += 32)
                if (rk[k] == RK_STALE) rk[k] = (k + 1 < m) ? pair_probe(tab, tok[k], tok[k + 1]) : TT_RANK_INF;
        }
        __syncwarp();
        for (u32 k = lane; k < m; k += 32) stage[a + k] = ext_id[tok[k]];
        if (lane == 0) piece_cnt[p] = m;
    }
}

// ---- K4, CTA per long piece (long whitespace / punctuation runs and other pieces > 256 bytes) -----
constexpr int LONG_THREADS = 1024;
constexpr u32 TOK_NEW = 0x80000000u;                  // token produced in the current round

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

// ---- K5a: token counts per block of pieces, then their exclusive prefix ---------------------------
constexpr int CNT_THREADS = 1024;

__global__ void __launch_bounds__(CNT_THREADS)
k_count(const u32* __restrict__ piece_cnt, TTHeader* hdr, u32* __restrict__ blk_cnt, unsigned long long ids_cap) {
    __shared__ u32 sc[40];
    __shared__ u32 s_islast;
    const u32 n_pieces = hdr->n_pieces;
    const bool dead = hdr->status != 0;
    const u32 p = blockIdx.x * CNT_THREADS + threadIdx.x;
    u32 v = (!dead && p < n_pieces) ? piece_cnt[p] : 0, tot;
    cta_excl_sum_scan(v, sc, &tot);
    if (threadIdx.x == 0) blk_cnt[blockIdx.x] = tot;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_islast = (atomicAdd(&hdr->count_done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!s_islast) return;
    __threadfence();
    const u32 nblk = gridDim.x;
    unsigned long long carry = 0;
    for (u32 b0 = 0; b0 < nblk; b0 += CNT_THREADS) {
        const u32 i = b0 + threadIdx.x;
        u32 x = i < nblk ? blk_cnt[i] : 0, t2;
        const u32 ex = cta_excl_sum_scan(x, sc, &t2);
        if (i < nblk) blk_cnt[i] = (u32)carry + ex;
        carry += t2;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        hdr->n_tokens = carry;
        if (!dead && carry > ids_cap) atomicMax(&hdr->status, 5 /* TT_ERR_CAPACITY */);
    }
}

// ---- K5b: token offsets per piece and coalesced scatter of the staged ids --------------------------
__global__ void __launch_bounds__(CNT_THREADS)
k_scatter(const u32* __restrict__ piece_off, const u32* __restrict__ piece_cnt, const u32* __restrict__ blk_base,
          const int32_t* __restrict__ stage, TTHeader* hdr, u32* __restrict__ tok_off, int32_t* __restrict__ ids_out,
          long long* __restrict__ count_out, int32_t* __restrict__ status_out) {
    __shared__ u32 sc[40];
    __shared__ u32 s_big[CNT_THREADS][3];
    __shared__ u32 s_nbig;
    const int status = hdr->status;
    const u32 n_pieces = hdr->n_pieces;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        if (status_out) *status_out = status;
        if (count_out) *count_out = status ? 0 : (long long)hdr->n_tokens;
        if (status || n_pieces == 0) tok_off[0] = 0;
    }
    if (status != 0) return;
    if (threadIdx.x == 0) s_nbig = 0;
    const u32 p = blockIdx.x * CNT_THREADS + threadIdx.x;
    const u32 c = p < n_pieces ? piece_cnt[p] : 0;
    u32 tot;
    const u32 dst = blk_base[blockIdx.x] + cta_excl_sum_scan(c, sc, &tot);
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
        for (u32 k = threadIdx.x; k < cc; k += CNT_THREADS) ids_out[d2 + k] = stage[src + k];
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

// C ABI of the toktier library (see include/toktier.h).  Host side: argument checks, vocabulary
// tables, workspace layout and the kernel chain  k_pretok<fused> (K1+K2, K3 per tile in shared memory, whole-piece
// lookups) -> k_merge (K4's merges, from the per-tile queues) -> k_scatter (K5); sessions
// (incremental repair), the added-token literal pass and the shadow verifier (host only) sit on top of it.
// Nothing here synchronises with the device except tt_vocab_load, tt_encode_host, tt_encode_timed and
// tt_session_append.
#include "../../include/toktier.h"
#include "tt_common.cuh"
#include "tt_pretok_kernels.cuh"
#include "tt_bpe.cuh"
#include "tt_spans.cuh"
#include "tt_session.cuh"
#include "tt_literals.cuh"
#include "unicode_table.inc"

#include <climits>
#include <mutex>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <unordered_map>
#include <unordered_set>
#include <atomic>
#include <vector>
#include <algorithm>

struct tt_vocab {
    int pattern = 0;
    int device = 0;
    int sm_count = 148;
    size_t n_merges = 0;
    uint4* d_slots = nullptr;
    u64* d_bytepair = nullptr;
    int32_t* d_ext_id = nullptr;
    u8* d_cls = nullptr;
    int cls_bytes = 0;
    PairTable tab{};
    TokSlot* d_tokslots = nullptr;
    TokTable toktab{};
    bool ignore_merges = false;
    LongSlot* d_longslots = nullptr; u8* d_longblob = nullptr;
    LongTable longtab{};
    size_t n_table_tokens = 0;
    uint2* d_meta = nullptr;             // per caller id: (byte length, non-continuation bytes) for tt_spans
    u32 meta_n = 0;
    LitEntry* d_lit_entries = nullptr; u8* d_lit_blob = nullptr;
    LitTable lit{};                      // added-token literals (tt_vocab_add_literals), n == 0: none
    u32 max_token_chars = 1;             // characters of the longest entry (stable boundary check of the sessions)
    // cached buffers of tt_encode_host
    u8* h_text = nullptr; int32_t* h_ids = nullptr; long long* h_scalars = nullptr; long long* h_scalars_dev = nullptr;
    u8* d_text = nullptr; int32_t* d_ids = nullptr; long long* d_count = nullptr; int32_t* d_status = nullptr;
    void* d_ws = nullptr; size_t host_cap = 0, ws_cap = 0;
    cudaStream_t host_stream = nullptr;
    cudaEvent_t slice_ev[8] = {};
};

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Epoch of a call: tags the status word of the workspace header (see TTHeader).  Never zero, never repeated.
static std::atomic<unsigned long long> g_epoch{1};
static inline unsigned long long next_epoch() { return g_epoch.fetch_add(1, std::memory_order_relaxed) & ((1ull << 56) - 1); }

extern "C" const char* tt_strerror(int code) {
    switch (code) {
        case TT_OK: return "ok";
        case TT_ERR_ARG: return "invalid argument";
        case TT_ERR_BAD_VOCAB: return "merge table rejected";
        case TT_ERR_CUDA: return "CUDA runtime error";
        case TT_ERR_INVALID_UTF8: return "input is not valid UTF-8";
        case TT_ERR_CAPACITY: return "output buffer too small";
        case TT_ERR_INTERNAL_TIMEOUT: return "bounded device loop gave up";
        case TT_ERR_TOO_LARGE: return "input exceeds the fixed limit of the no-allocation entry point";
        case TT_ERR_BAD_IDS: return "token ids do not belong to this vocabulary or do not spell a text of the given length";
        default: return "unknown code";
    }
}

extern "C" size_t tt_class_table(uint8_t* out, size_t cap) {
    const size_t n = 0x110000;
    for (size_t cp = 0; cp < n && cp < cap; cp++) {
        unsigned v = tt_cls_stage2_host[(size_t)tt_cls_stage1_host[cp >> 8] * 128 + ((cp & 0xFF) >> 1)];
        out[cp] = (uint8_t)((cp & 1) ? (v >> 4) : (v & 15));
    }
    return n;
}

extern "C" void tt_vocab_free(tt_vocab* v) {
    if (!v) return;
    cudaFree(v->d_slots); cudaFree(v->d_bytepair); cudaFree(v->d_ext_id); cudaFree(v->d_cls); cudaFree(v->d_lit_entries); cudaFree(v->d_lit_blob); cudaFree(v->d_tokslots); cudaFree(v->d_longslots); cudaFree(v->d_longblob); cudaFree(v->d_meta);
    cudaFree(v->d_text); cudaFree(v->d_ids); cudaFree(v->d_count); cudaFree(v->d_status); cudaFree(v->d_ws);
    if (v->h_text) cudaFreeHost(v->h_text);
    if (v->h_ids) cudaFreeHost(v->h_ids);
    if (v->h_scalars) cudaFreeHost(v->h_scalars);
    if (v->host_stream) cudaStreamDestroy(v->host_stream);
    for (cudaEvent_t e : v->slice_ev) if (e) cudaEventDestroy(e);
    delete v;
}


// Whole-piece table: every token of at most TT_TOKTAB_MAXLEN bytes is encoded with the merge kernel
// itself; those whose byte string yields exactly that one token are entered (key = bytes, value = the
// caller's id).  A hit in the table therefore equals what the merge loop returns for that piece.
// With ignore_merges every entry is entered as it is (the first entry that spells given bytes wins) and
// entries longer than TT_TOKTAB_MAXLEN bytes go to the long-entry table.
static int build_token_table(tt_vocab* v, const tt_merge* merges, size_t n_merges, const std::vector<int32_t>& ext_id) {
    (void)merges;
    // byte strings of the merge results, by internal id (operands are lower internal ids by construction)
    std::vector<std::string> bytes(256 + n_merges);
    for (int b = 0; b < 256; b++) bytes[b] = std::string(1, (char)b);
    std::unordered_map<int32_t, u32> internal;
    internal.reserve(2 * ext_id.size());
    for (size_t i = 0; i < ext_id.size(); i++) internal.emplace(ext_id[i], (u32)i);
    std::vector<u32> cand;                       // internal ids of candidate tokens
    std::vector<u32> longer;                     // ignore_merges: internal ids of entries beyond TT_TOKTAB_MAXLEN bytes
    std::unordered_set<std::string> spelled;     // ignore_merges: byte strings seen so far (base bytes first)
    if (v->ignore_merges) for (int b = 0; b < 256; b++) spelled.insert(bytes[b]);
    std::vector<u8> cat; std::vector<u32> off;
    for (size_t r = 0; r < n_merges; r++) {
        const std::string& L = bytes[internal[merges[r].left]];
        const std::string& R = bytes[internal[merges[r].right]];
        if (L.size() + R.size() <= 4096) bytes[256 + r] = L + R;          // longer strings are never candidates
        else bytes[256 + r] = std::string(4097, 'x');
        const std::string& t = bytes[256 + r];
        if (v->ignore_merges && t.size() > 4096) return TT_ERR_BAD_VOCAB;   // documented limit of the whole-piece rule
        if (v->ignore_merges && !spelled.insert(t).second) continue;      // an earlier entry spells the same bytes
        if (v->ignore_merges && t.size() > (size_t)TT_TOKTAB_MAXLEN) longer.push_back((u32)(256 + r));
        if (t.size() >= 2 && t.size() <= (size_t)TT_TOKTAB_MAXLEN) {
            cand.push_back((u32)(256 + r)); off.push_back((u32)cat.size());
            cat.insert(cat.end(), t.begin(), t.end());
        }
    }
    off.push_back((u32)cat.size());
    if (!longer.empty()) {
        u32 cap = 64;
        while (cap < 2 * longer.size() + 2) cap <<= 1;
        std::vector<LongSlot> ls(cap);
        memset(ls.data(), 0, cap * sizeof(LongSlot));
        std::vector<u8> blob;
        u32 maxlen = 0;
        for (u32 t : longer) {
            const std::string& b = bytes[t];
            const u64 hsh = longtab_hash((const u8*)b.data(), (u32)b.size());
            u32 sl = (u32)(hsh >> 32) & (cap - 1);
            while (ls[sl].len != 0) sl = (sl + 1) & (cap - 1);
            ls[sl].hash = hsh; ls[sl].off = (u32)blob.size(); ls[sl].len = (u32)b.size(); ls[sl].id = ext_id[t];
            blob.insert(blob.end(), b.begin(), b.end());
            maxlen = maxlen > (u32)b.size() ? maxlen : (u32)b.size();
        }
        if (cudaMalloc(&v->d_longslots, cap * sizeof(LongSlot)) != cudaSuccess || cudaMalloc(&v->d_longblob, blob.size() + 16) != cudaSuccess ||
            cudaMemcpy(v->d_longslots, ls.data(), cap * sizeof(LongSlot), cudaMemcpyHostToDevice) != cudaSuccess ||
            cudaMemcpy(v->d_longblob, blob.data(), blob.size(), cudaMemcpyHostToDevice) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
        v->longtab.slots = v->d_longslots; v->longtab.blob = v->d_longblob; v->longtab.mask = cap - 1; v->longtab.maxlen = maxlen;
    }
    if (cand.empty()) return TT_OK;
    const size_t nb = cat.size(), np = cand.size();
    std::vector<u32> keep;
    if (v->ignore_merges) { for (size_t i = 0; i < np; i++) keep.push_back((u32)i); }
    else {
    // the per-tile records of the concatenation as the first kernel would leave them without a table: every piece
    // but the last of its tile is queued (all are short), the last one of every tile is k_merge's anyway
    const size_t nchunks = (nb + TT_CHUNK - 1) / TT_CHUNK, ntiles = (nchunks + TT_TILE_CHUNKS - 1) / TT_TILE_CHUNKS;
    std::vector<u32> tile_base(ntiles + 1, 0), tile_cnt(ntiles, 0), tile_first(ntiles, TT_NONE), tile_last(ntiles, TT_NONE), tile_q(ntiles, 0);
    std::vector<u16> off16(ntiles * TT_TILE_BYTES, 0);
    std::vector<u32> qv(ntiles * TT_TILE_QCAP, 0);
    for (size_t i = 0; i < np; i++) {
        const size_t t = off[i] / TT_TILE_BYTES; const u32 o = off[i] % TT_TILE_BYTES;
        off16[t * TT_TILE_BYTES + tile_cnt[t]] = (u16)o;
        if (tile_first[t] == TT_NONE) tile_first[t] = o;
        tile_last[t] = o; tile_cnt[t]++;
    }
    for (size_t t = 0; t < ntiles; t++) tile_base[t + 1] = tile_base[t] + tile_cnt[t];
    for (size_t t = 0; t < ntiles; t++)
        for (u32 k = 0; k + 1 < tile_cnt[t]; k++) {
            const size_t i = tile_base[t] + k;
            qv[t * TT_TILE_QCAP + tile_q[t]++] = off16[t * TT_TILE_BYTES + k] | (k << 11) | ((off[i + 1] - off[i] - 1) << 22);
        }
    u8* d_text = nullptr; u32 *d_tc = nullptr, *d_tf = nullptr, *d_tl = nullptr, *d_tq = nullptr, *d_cnt = nullptr, *d_tt = nullptr, *d_q = nullptr; u16 *d_o16 = nullptr, *d_lg = nullptr; int32_t* d_stage = nullptr;
    TTHeader* d_hdr = nullptr;
    std::vector<u32> cnt(ntiles * TT_TILE_BYTES); std::vector<int32_t> stage(nb);
    auto up = [&](auto** dp, const auto& h) {
        return cudaMalloc(dp, h.size() * sizeof(h[0]) + 64) == cudaSuccess && cudaMemcpy(*dp, h.data(), h.size() * sizeof(h[0]), cudaMemcpyHostToDevice) == cudaSuccess;
    };
    bool ok = cudaMalloc(&d_text, nchunks * TT_CHUNK + 64) == cudaSuccess && cudaMemcpy(d_text, cat.data(), nb, cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && up(&d_tc, tile_cnt) && up(&d_tf, tile_first) && up(&d_tl, tile_last) && up(&d_tq, tile_q) && up(&d_o16, off16) && up(&d_q, qv);
    ok = ok && cudaMalloc(&d_lg, ntiles * TT_TILE_LONGCAP * sizeof(u16)) == cudaSuccess && cudaMalloc(&d_tt, (ntiles + 1) * sizeof(u32)) == cudaSuccess &&
              cudaMalloc(&d_cnt, cnt.size() * sizeof(u32)) == cudaSuccess && cudaMalloc(&d_stage, (nb + 1) * sizeof(int32_t)) == cudaSuccess &&
              cudaMalloc(&d_hdr, sizeof(TTHeader)) == cudaSuccess;
    ok = ok && cudaMemset(d_hdr, 0, sizeof(TTHeader)) == cudaSuccess && cudaMemset(d_tt, 0, (ntiles + 1) * sizeof(u32)) == cudaSuccess;
    if (ok) {
        PieceParams Q;
        Q.base = d_text; Q.shift = 0; Q.hi = (long long)nb; Q.ntiles = (int)ntiles;
        Q.tile_cnt = d_tc; Q.tile_first = d_tf; Q.tile_last = d_tl; Q.tile_q = d_tq; Q.tile_long = d_lg; Q.piece_off16 = d_o16; Q.q = d_q;
        Q.hdr = d_hdr; Q.epoch = next_epoch(); Q.tab = v->tab;
        Q.toktab.slots = nullptr; Q.toktab.mask = 0; Q.toktab.shift = 0;      // no table yet: every piece is merged
        Q.longtab = LongTable{}; Q.litstart = nullptr;
        Q.ext_id = v->d_ext_id; Q.piece_cnt = d_cnt; Q.stage = d_stage; Q.pairbuf = nullptr; Q.tile_tok = d_tt; Q.grp_tok = nullptr; Q.wq = nullptr; Q.gq = nullptr; Q.gq_x[0] = Q.gq_x[1] = Q.gq_x[2] = nullptr; Q.lq = nullptr;
        k_merge<<<v->sm_count * MERGE_CTAS_PER_SM, MERGE_THREADS, MERGE_SMEM_BYTES>>>(Q);
        ok = cudaGetLastError() == cudaSuccess && cudaDeviceSynchronize() == cudaSuccess;
    }
    ok = ok && cudaMemcpy(cnt.data(), d_cnt, cnt.size() * sizeof(u32), cudaMemcpyDeviceToHost) == cudaSuccess;
    ok = ok && cudaMemcpy(stage.data(), d_stage, nb * sizeof(int32_t), cudaMemcpyDeviceToHost) == cudaSuccess;
    cudaFree(d_text); cudaFree(d_tc); cudaFree(d_tf); cudaFree(d_tl); cudaFree(d_tq); cudaFree(d_o16); cudaFree(d_q); cudaFree(d_lg); cudaFree(d_tt); cudaFree(d_cnt); cudaFree(d_stage); cudaFree(d_hdr);
    if (!ok) { cudaGetLastError(); return TT_ERR_CUDA; }
    for (size_t i = 0; i < np; i++) {
        const size_t tile = off[i] / TT_TILE_BYTES, slot = tile * TT_TILE_BYTES + (i - tile_base[tile]);   // pieces are indexed per tile
        if ((int32_t)cnt[slot] == -1 && stage[off[i]] == ext_id[cand[i]]) keep.push_back((u32)i);           // minus the staged count
    }
    }
    u32 cap = 1024;
    while (cap < 2 * keep.size() + 2) cap <<= 1;
    u32 log2cap = 0;
    while ((1u << log2cap) < cap) log2cap++;
    const u32 mask = cap - 1, shift = 32 - log2cap;
    std::vector<TokSlot> slots(cap);
    memset(slots.data(), 0, cap * sizeof(TokSlot));
    for (u32 i : keep) {
        const u32 n = off[i + 1] - off[i];
        u8 key[24] = {0};
        memcpy(key, cat.data() + off[i], n);
        u32 k[6]; memcpy(k, key, 24);
        u32 hh = toktab_hash_final(toktab_hash_rest(toktab_hash_short(k[0], k[1], n), k[2], k[3], k[4], k[5]), shift);
        while (slots[hh].len != 0) hh = (hh + 1) & mask;
        slots[hh].len = n; slots[hh].id = ext_id[cand[i]];
        for (int j = 0; j < 6; j++) slots[hh].k[j] = k[j];
    }
    if (cudaMalloc(&v->d_tokslots, (size_t)cap * sizeof(TokSlot)) != cudaSuccess ||
        cudaMemcpy(v->d_tokslots, slots.data(), (size_t)cap * sizeof(TokSlot), cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError(); return TT_ERR_CUDA;
    }
    v->toktab.slots = v->d_tokslots; v->toktab.mask = mask; v->toktab.shift = shift;
    v->n_table_tokens = keep.size();
    return TT_OK;
}

extern "C" size_t tt_vocab_table_entries(const tt_vocab* v) { return v ? v->n_table_tokens : 0; }

extern "C" int tt_vocab_load(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256], int pattern_id,
                             tt_vocab** out) {
    return tt_vocab_load_ex(merges, n_merges, byte_map, pattern_id, 0u, out);
}

// ---- ranks and guards of the pairs (host only, no CUDA call) ---------------------------------------------------
// For every merge (a, b) of rank r: the pair (a, b) gets the rank; every pair (u, b) with u on the right spine
// of a's merge tree gets cl <= r (the merge can take b from the left of a token built on u); every pair (a, w)
// with w on the left spine of b gets cr <= r.  Ranks ascend, so the first value written is the lowest.
struct PairTriple { u32 r, cl, cr; };
static int build_pair_info(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256],
                           std::unordered_map<int32_t, u32>& internal, std::vector<int32_t>& ext_id,
                           std::unordered_map<u64, PairTriple>& info) {
    if (n_merges > TT_MAX_INTERNAL - 256) return TT_ERR_ARG;
    // external id -> internal id (byte b -> b, result of rank r -> 256 + r)
    internal.clear(); internal.reserve(512 + 2 * n_merges);
    ext_id.assign(256 + n_merges, 0);
    for (int b = 0; b < 256; b++) {
        if (byte_map[b] < 0 || !internal.emplace(byte_map[b], (u32)b).second) return TT_ERR_BAD_VOCAB;   // not injective
        ext_id[b] = byte_map[b];
    }
    std::vector<u32> lch(256 + n_merges, 0xFFFFFFFFu), rch(256 + n_merges, 0xFFFFFFFFu);   // children of every merge result
    const PairTriple none{TT_RANK_INF, TT_RANK_INF, TT_RANK_INF};
    info.clear(); info.reserve(6 * n_merges + 16);
    for (size_t r = 0; r < n_merges; r++) {
        const tt_merge& m = merges[r];
        auto l = internal.find(m.left), rr = internal.find(m.right);
        if (l == internal.end() || rr == internal.end()) return TT_ERR_BAD_VOCAB;      // operand not yet defined
        if (m.result < 0 || internal.count(m.result)) return TT_ERR_BAD_VOCAB;         // result id reused
        const u32 a = l->second, b = rr->second;
        auto ins = info.emplace(((u64)a << TT_ID_BITS) | b, none);
        if (ins.first->second.r != TT_RANK_INF) return TT_ERR_BAD_VOCAB;               // duplicate pair
        ins.first->second.r = (u32)r;
        lch[256 + r] = a; rch[256 + r] = b;
        for (u32 u = a; u != 0xFFFFFFFFu; u = u >= 256 ? rch[u] : 0xFFFFFFFFu) {
            PairTriple& t = info.emplace(((u64)u << TT_ID_BITS) | b, none).first->second;
            if (t.cl == TT_RANK_INF) t.cl = (u32)r;
        }
        for (u32 w = b; w != 0xFFFFFFFFu; w = w >= 256 ? lch[w] : 0xFFFFFFFFu) {
            PairTriple& t = info.emplace(((u64)a << TT_ID_BITS) | w, none).first->second;
            if (t.cr == TT_RANK_INF) t.cr = (u32)r;
        }
        internal.emplace(m.result, (u32)(256 + r));
        ext_id[256 + r] = m.result;
    }
    return TT_OK;
}

extern "C" int tt_pair_info_host(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256],
                                 const int32_t* left, const int32_t* right, size_t n_pairs, int64_t* out) {
    if (!byte_map || (n_merges && !merges) || (n_pairs && (!left || !right || !out))) return TT_ERR_ARG;
    std::unordered_map<int32_t, u32> internal;
    std::vector<int32_t> ext_id;
    std::unordered_map<u64, PairTriple> info;
    const int rc = build_pair_info(merges, n_merges, byte_map, internal, ext_id, info);
    if (rc != TT_OK) return rc;
    for (size_t i = 0; i < n_pairs; i++) {
        PairTriple t{TT_RANK_INF, TT_RANK_INF, TT_RANK_INF};
        auto l = internal.find(left[i]), r = internal.find(right[i]);
        if (l != internal.end() && r != internal.end()) {
            auto it = info.find(((u64)l->second << TT_ID_BITS) | r->second);
            if (it != info.end()) t = it->second;
        }
        out[3 * i] = t.r == TT_RANK_INF ? -1 : (int64_t)t.r;
        out[3 * i + 1] = t.cl == TT_RANK_INF ? -1 : (int64_t)t.cl;
        out[3 * i + 2] = t.cr == TT_RANK_INF ? -1 : (int64_t)t.cr;
    }
    return TT_OK;
}

extern "C" int tt_vocab_load_ex(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256], int pattern_id,
                                unsigned flags, tt_vocab** out) {
    if (out) *out = nullptr;
    if (!out || !byte_map || (n_merges && !merges) || (flags & ~TT_VOCAB_IGNORE_MERGES)) return TT_ERR_ARG;
    if (pattern_id != TT_PATTERN_CL100K && pattern_id != TT_PATTERN_O200K && pattern_id != TT_PATTERN_CL100K_N1 && pattern_id != TT_PATTERN_SPLIT3) return TT_ERR_ARG;
    std::unordered_map<int32_t, u32> internal;
    std::vector<int32_t> ext_id;
    std::unordered_map<u64, PairTriple> info;           // key (left << 18 | right) -> rank and guards
    { const int rc = build_pair_info(merges, n_merges, byte_map, internal, ext_id, info); if (rc != TT_OK) return rc; }
    // pair table: two-choice hashing, buckets of two 16-byte slots, at most half of the slots used
    std::vector<u64> bytepair(65536, ~0ull);            // the byte-byte pairs, directly indexed: three 20-bit fields
    std::vector<uint4> entries;
    entries.reserve(info.size());
    for (const auto& kv : info) {
        const u64 key = kv.first;
        const PairTriple& t = kv.second;
        const u32 a = (u32)(key >> TT_ID_BITS), b = (u32)(key & (TT_MAX_INTERNAL - 1));
        if (a < 256 && b < 256)
            bytepair[(a << 8) | b] = (u64)f20_encode(t.r) | ((u64)f20_encode(t.cl) << 20) | ((u64)f20_encode(t.cr) << 40);
        const u64 kr = (key << 20) | f20_encode(t.r);
        entries.push_back(make_uint4((u32)kr, (u32)(kr >> 32), t.cl, t.cr));
    }
    u32 nbuckets = 256;
    while (nbuckets < entries.size() + 1) nbuckets <<= 1;
    std::vector<uint4> slots;
    u32 mask = 0, shift = 0;
    size_t cap = 0;
    for (;; nbuckets <<= 1) {                            // a placement that fails (not seen so far) doubles the table
        if (nbuckets > (1u << 24)) return TT_ERR_BAD_VOCAB;
        u32 log2b = 0;
        while ((1u << log2b) < nbuckets) log2b++;
        mask = nbuckets - 1; shift = 32 - log2b; cap = 2 * (size_t)nbuckets;
        slots.assign(cap, make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu));
        auto is_free = [](const uint4& s) { return (s.x & s.y) == 0xFFFFFFFFu; };
        auto key_of = [](const uint4& s) { return (((u64)s.y << 32) | s.x) >> 20; };
        u64 rng = 0x9E3779B97F4A7C15ull;
        bool ok_all = true;
        for (const uint4& e0 : entries) {
            uint4 cur = e0;
            u32 avoid = 0xFFFFFFFFu;                     // do not move straight back into the bucket just left
            bool placed = false;
            for (int iter = 0; iter < 2000 && !placed; iter++) {
                const u64 key = key_of(cur);
                const u32 h0 = pair_bucket(key, shift), h1 = pair_bucket_alt(key, shift, h0);
                for (u32 h : {h0, h1}) {
                    uint4* bk = &slots[2 * (size_t)h];
                    for (int k = 0; k < 2 && !placed; k++) if (is_free(bk[k])) { bk[k] = cur; placed = true; }
                    if (placed) break;
                }
                if (placed) break;
                rng = rng * 6364136223846793005ull + 1442695040888963407ull;
                const u32 h = (h0 == avoid) ? h1 : (h1 == avoid) ? h0 : ((rng >> 33) & 1 ? h1 : h0);
                uint4* bk = &slots[2 * (size_t)h + ((rng >> 40) & 1)];
                const uint4 victim = *bk;
                *bk = cur; cur = victim; avoid = h;
            }
            if (!placed) { ok_all = false; break; }
        }
        if (ok_all) break;
    }
    tt_vocab* v = new (std::nothrow) tt_vocab();
    if (!v) return TT_ERR_CUDA;
    v->pattern = pattern_id; v->n_merges = n_merges; v->ignore_merges = (flags & TT_VOCAB_IGNORE_MERGES) != 0;
    // class tables: stage1 | stage2 | ascii
    const int stage2_bytes = TT_CLS_NBLOCKS * 128;
    v->cls_bytes = (int)align_up(0x1100 + stage2_bytes, 16) + 128;
    std::vector<u8> cls(v->cls_bytes, 0);
    memcpy(cls.data(), tt_cls_stage1_host, 0x1100);
    memcpy(cls.data() + 0x1100, tt_cls_stage2_host, stage2_bytes);
    tt_fill_ascii_table(cls.data() + v->cls_bytes - 128);
    bool ok = cudaGetDevice(&v->device) == cudaSuccess;
    ok = ok && cudaDeviceGetAttribute(&v->sm_count, cudaDevAttrMultiProcessorCount, v->device) == cudaSuccess;
    ok = ok && cudaMalloc(&v->d_slots, cap * sizeof(uint4)) == cudaSuccess;
    ok = ok && cudaMalloc(&v->d_bytepair, bytepair.size() * sizeof(u64)) == cudaSuccess;
    ok = ok && cudaMemcpy(v->d_bytepair, bytepair.data(), bytepair.size() * sizeof(u64), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMalloc(&v->d_ext_id, ext_id.size() * sizeof(int32_t)) == cudaSuccess;
    ok = ok && cudaMalloc(&v->d_cls, v->cls_bytes) == cudaSuccess;
    ok = ok && cudaMemcpy(v->d_slots, slots.data(), cap * sizeof(uint4), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(v->d_ext_id, ext_id.data(), ext_id.size() * sizeof(int32_t), cudaMemcpyHostToDevice) == cudaSuccess;
    ok = ok && cudaMemcpy(v->d_cls, cls.data(), v->cls_bytes, cudaMemcpyHostToDevice) == cudaSuccess;
    if (!ok) { cudaGetLastError(); tt_vocab_free(v); return TT_ERR_CUDA; }
    v->tab.slots = v->d_slots; v->tab.bytepair = v->d_bytepair; v->tab.mask = mask; v->tab.shift = shift;
    if (cudaFuncSetAttribute(k_merge, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MERGE_SMEM_BYTES) != cudaSuccess ||
        cudaFuncSetAttribute(k_merge_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)MERGE_SMEM_BYTES) != cudaSuccess) { cudaGetLastError(); tt_vocab_free(v); return TT_ERR_CUDA; }
    { const int rc = build_token_table(v, merges, n_merges, ext_id); if (rc != TT_OK) { tt_vocab_free(v); return rc; } }
    {   // byte length and number of non-continuation bytes of every token, indexed by the caller's id
        std::vector<uint2> in(256 + n_merges);
        for (int b = 0; b < 256; b++) in[b] = make_uint2(1u, (b & 0xC0) != 0x80 ? 1u : 0u);
        int32_t max_ext = 0;
        for (int32_t e : ext_id) max_ext = e > max_ext ? e : max_ext;
        for (size_t r = 0; r < n_merges; r++) {
            const uint2 L = in[internal[merges[r].left]], R = in[internal[merges[r].right]];
            in[256 + r] = make_uint2(L.x + R.x, L.y + R.y);
            if (in[256 + r].y > v->max_token_chars) v->max_token_chars = in[256 + r].y;
        }
        if (max_ext < (1 << 24)) {
            std::vector<uint2> meta((size_t)max_ext + 1, make_uint2(0, 0));
            for (size_t i = 0; i < ext_id.size(); i++) meta[ext_id[i]] = in[i];
            if (cudaMalloc(&v->d_meta, meta.size() * sizeof(uint2)) != cudaSuccess ||
                cudaMemcpy(v->d_meta, meta.data(), meta.size() * sizeof(uint2), cudaMemcpyHostToDevice) != cudaSuccess) {
                cudaGetLastError(); tt_vocab_free(v); return TT_ERR_CUDA;
            }
            v->meta_n = (u32)meta.size();
        }
    }
    *out = v;
    return TT_OK;
}

// ---- workspace layout ----------------------------------------------------------------------------
static size_t carve(TTWorkspace* w, void* base, size_t max_len, size_t max_docs) {
    (void)max_docs;
    const size_t padded = max_len + 64;                       // aligned frame: up to 15 bytes of shift + tail
    const size_t nchunks = padded / TT_CHUNK + 2;
    const size_t ntiles = nchunks / TT_TILE_CHUNKS + 2;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return (char*)base + o; };
    char* p;
    p = take(sizeof(TTHeader));                 if (w) w->hdr = (TTHeader*)p;
    p = take((padded / 32 + 4) * sizeof(u32));  if (w) w->docmask = (u32*)p;
    p = take(nchunks * sizeof(u16));            if (w) w->startmask = (u16*)p;
    p = take((ntiles + 1) * sizeof(u32));       if (w) w->tile_cnt = (u32*)p;
    p = take((ntiles + 1) * sizeof(u32));       if (w) w->tile_first = (u32*)p;
    p = take((ntiles + 1) * sizeof(u32));       if (w) w->tile_last = (u32*)p;
    p = take((ntiles + 1) * sizeof(u32));       if (w) w->tile_tok = (u32*)p;
    p = take((ntiles + 1) * sizeof(u32));       if (w) w->tile_q = (u32*)p;
    p = take((ntiles / TT_GROUP_TILES + 2) * sizeof(u32));   if (w) w->grp_tok = (u32*)p;
    p = take(ntiles * TT_TILE_LONGCAP * sizeof(u16));        if (w) w->tile_long = (u16*)p;
    p = take(ntiles * TT_TILE_BYTES * sizeof(u16));          if (w) w->piece_off16 = (u16*)p;
    p = take(ntiles * TT_TILE_BYTES * sizeof(u32));          if (w) w->piece_cnt = (u32*)p;
    p = take(ntiles * TT_TILE_QCAP * sizeof(u32));           if (w) w->q = (u32*)p;
    // the global lists of bulk text: only where a text can have more tiles than a request's job search covers (any
    // alignment of the text counted in)
    const bool bulk_lists = (15 + max_len + TT_TILE_BYTES - 1) / TT_TILE_BYTES > (size_t)MERGE_SR_MAX_TILES;
    if (w) { w->wq = nullptr; w->gq = nullptr; w->lq = nullptr; for (int c = 0; c < TT_SHORT_CLASSES - 1; c++) w->gq_x[c] = nullptr; }
    if (bulk_lists) {
        p = take((max_len / 33 + 64) * sizeof(u64));             if (w) w->wq = (u64*)p;
        p = take((max_len / 2 + 64) * sizeof(u64));              if (w) w->gq = (u64*)p;
        for (int c = 1; c < TT_SHORT_CLASSES; c++) {              // a piece of class c has more bytes than class c - 1 allows
            p = take((max_len / (tt_short_class_max(c - 1) + 1) + 64) * sizeof(u64));   if (w) w->gq_x[c - 1] = (u64*)p;
        }
        p = take((max_len / 257 + 16) * sizeof(uint4));          if (w) w->lq = (uint4*)p;
    }
    p = take((max_len + 1) * sizeof(int32_t));  if (w) w->stage = (int32_t*)p;
    p = take((max_len + 1) * sizeof(u64));      if (w) w->pairbuf = (u64*)p;
    p = take(padded + 16);                      if (w) w->cand = (u8*)p;
    p = take((padded / 32 + 4) * sizeof(u32));  if (w) w->litstart = (u32*)p;
    p = take((padded / 32 + 4) * sizeof(u32));  if (w) w->litin = (u32*)p;
    p = take((padded / 32 + 4) * sizeof(u32));  if (w) w->cutmask = (u32*)p;
    return off;
}

extern "C" size_t tt_workspace_bytes(const tt_vocab* v, size_t max_len, size_t max_docs) {
    (void)v;
    return carve(nullptr, nullptr, max_len, max_docs);
}

#define CK(x) do { if ((x) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; } } while (0)

// One instance of the first kernel per pattern (the pattern's rules are compiled in), chosen here.
template <bool FUSED, int MINB>
static void launch_pretok(int grid, cudaStream_t st, const PretokParams& P, const FrontParams& F) {
    const size_t smem = TT_PRETOK_SMEM_BYTES;
    switch (P.pattern) {
    case TT_PATTERN_O200K:     k_pretok<FUSED, MINB, TT_PATTERN_O200K><<<grid, TT_TILE_CHUNKS, smem, st>>>(P, F); break;
    case TT_PATTERN_CL100K_N1: k_pretok<FUSED, MINB, TT_PATTERN_CL100K_N1><<<grid, TT_TILE_CHUNKS, smem, st>>>(P, F); break;
    case TT_PATTERN_CUTS:      if constexpr (!FUSED) k_pretok<false, MINB, TT_PATTERN_CUTS><<<grid, TT_TILE_CHUNKS, smem, st>>>(P, F); break;
    default:                   k_pretok<FUSED, MINB, TT_PATTERN_CL100K><<<grid, TT_TILE_CHUNKS, smem, st>>>(P, F); break;
    }
}

// Enqueues K1+K2 (and K3 when piece_off_dst is given: only tt_pretokenize materialises the offsets;
// the encode chain derives them per tile from the start flags).
static int run_pretok(const tt_vocab* v, const uint8_t* text, size_t len, const int64_t* doc_off, size_t n_docs,
                      cudaStream_t st, TTWorkspace& w, u32* piece_off_dst, PretokParams& P, bool literals = false, bool fused = false,
                      const uint8_t* host_src = nullptr) {
    const uintptr_t addr = (uintptr_t)text;
    const long long shift = (long long)(addr & 15);
    P.base = (const u8*)(addr - shift);
    P.src = nullptr; P.copy = nullptr;
    if (host_src) {                                           // pinned host text, read by the first kernel itself (tt_encode_host)
        if ((long long)((uintptr_t)host_src & 15) != shift) return TT_ERR_ARG;     // the device copy shares the host text's 16-byte frame
        P.src = host_src - shift; P.copy = (u8*)(addr - shift);
    }
    P.lo = shift; P.hi = shift + (long long)len;
    P.nchunks = (P.hi + TT_CHUNK - 1) / TT_CHUNK;
    P.ntiles = (int)((P.nchunks + TT_TILE_CHUNKS - 1) / TT_TILE_CHUNKS);
    P.pattern = v->pattern; P.epoch = next_epoch();
    P.docmask = nullptr; P.litstart = nullptr; P.litin = nullptr;
    P.startmask = w.startmask; P.tile_cnt = w.tile_cnt; P.tile_first = w.tile_first; P.want_prefix = piece_off_dst != nullptr; P.hdr = w.hdr;
    P.cls_tables = v->d_cls; P.cls_bytes = v->cls_bytes;
    if (doc_off) {
        CK(cudaMemsetAsync(w.docmask, 0, ((size_t)P.hi / 32 + 4) * sizeof(u32), st));
        const int threads = 256, blocks = (int)((n_docs + 1 + threads - 1) / threads);
        k_docmask<<<blocks, threads, 0, st>>>((const long long*)doc_off, (int)n_docs, shift, (long long)len, w.docmask, w.hdr, P.epoch);
        P.docmask = w.docmask;
    }
    if (literals && !doc_off) {
        // added-token literal pass: extracted literals become documents of their own and single pieces
        const size_t words = ((size_t)P.hi / 32 + 4) * sizeof(u32);
        CK(cudaMemsetAsync(w.docmask, 0, words, st));
        CK(cudaMemsetAsync(w.litstart, 0, words, st));
        CK(cudaMemsetAsync(w.litin, 0, words, st));
        LitParams L;
        L.base = P.base; L.lo = P.lo; L.hi = P.hi; L.tab = v->lit; L.cand = w.cand; L.stage = w.stage;
        L.docmask = w.docmask; L.litstart = w.litstart; L.litin = w.litin;
        const size_t want = (len + 255) / 256;
        const int lgrid = (int)(want < (size_t)v->sm_count * 8 ? want : (size_t)v->sm_count * 8);
        k_lit_scan<<<lgrid, 256, 0, st>>>(L);
        k_lit_select<<<lgrid, 256, 0, st>>>(L);
        P.docmask = w.docmask; P.litstart = w.litstart; P.litin = w.litin;
    }
    const bool bulk = P.ntiles > MERGE_SR_MAX_TILES;
    const int per_sm = bulk && fused ? PRETOK_CTAS_BULK : PRETOK_CTAS_REQUEST;
    const int grid = P.ntiles < v->sm_count * per_sm ? P.ntiles : v->sm_count * per_sm;
    if (v->pattern == TT_PATTERN_SPLIT3) {
        // stages A and B: span starts into cutmask (with the caller's document starts); stage C: pattern 0 with
        // those cuts as its document boundaries
        PretokParams C1 = P;
        C1.pattern = TT_PATTERN_CUTS; C1.startmask = reinterpret_cast<u16*>(w.cutmask);
        C1.want_prefix = 0; C1.litstart = nullptr; C1.litin = nullptr;
        launch_pretok<false, PRETOK_CTAS_REQUEST>(grid, st, C1, FrontParams{});
        P.pattern = TT_PATTERN_CL100K; P.docmask = w.cutmask;
    }
    if (fused) {
        FrontParams F;
        F.tile_last = w.tile_last; F.tile_tok = w.tile_tok; F.tile_q = w.tile_q; F.tile_long = w.tile_long; F.piece_off16 = w.piece_off16;
        F.piece_cnt = w.piece_cnt; F.q = w.q; F.toktab = v->toktab; F.longtab = v->longtab; F.ext_id = v->d_ext_id;
        F.wq = P.ntiles > MERGE_SR_MAX_TILES ? w.wq : nullptr;
        if (bulk) launch_pretok<true, PRETOK_CTAS_BULK>(grid, st, P, F);
        else launch_pretok<true, PRETOK_CTAS_REQUEST>(grid, st, P, F);
    } else launch_pretok<false, PRETOK_CTAS_REQUEST>(grid, st, P, FrontParams{});
    if (piece_off_dst)
        k_compact<<<grid, TT_TILE_CHUNKS, 0, st>>>(w.startmask, w.tile_cnt, P.nchunks, P.ntiles, shift, (long long)len,
                                                   piece_off_dst, w.hdr, P.epoch);
    CK(cudaGetLastError());
    return TT_OK;
}

static int check_common(const tt_vocab* v, const void* text, size_t len, void* workspace, size_t workspace_bytes,
                        size_t n_docs) {
    if (!v || !workspace || (len && !text)) return TT_ERR_ARG;
    if (len >= (size_t)INT32_MAX - 64) return TT_ERR_ARG;
    if (((uintptr_t)workspace & 255) != 0) return TT_ERR_ARG;
    if (workspace_bytes < tt_workspace_bytes(v, len, n_docs)) return TT_ERR_ARG;
    return TT_OK;
}

// Launches `kernel` so that it may begin while the kernel before it on the stream is still draining
// (programmatic dependent launch): its CTAs are placed as soon as every CTA of the predecessor has
// signalled, and wait inside the kernel (cudaGridDependencySynchronize) until the predecessor's memory
// is complete.  Only the launch latency is hidden; the data dependence is unchanged.
template <typename Params>
static cudaError_t launch_after(void (*kernel)(const Params), int grid, int block, cudaStream_t st, const Params& p, size_t smem = 0) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid); cfg.blockDim = dim3((unsigned)block); cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

static int encode_impl(const tt_vocab* v, const uint8_t* text, size_t len, const int64_t* doc_off, size_t n_docs,
                       cudaStream_t st, int32_t* ids_out, size_t ids_cap, int64_t* count_out, int64_t* ids_off_out,
                       int32_t* status_out, void* workspace, cudaEvent_t* ev = nullptr, bool literals = false,
                       const uint8_t* host_src = nullptr) {
#define MARK(i) do { if (ev) cudaEventRecord(ev[i], st); } while (0)
    TTWorkspace w;
    carve(&w, workspace, len, n_docs);
    if (len == 0) {
        if (count_out) CK(cudaMemsetAsync(count_out, 0, sizeof(int64_t), st));
        if (ids_off_out) CK(cudaMemsetAsync(ids_off_out, 0, (n_docs + 1) * sizeof(int64_t), st));
        CK(cudaMemsetAsync(status_out, 0, sizeof(int32_t), st));
        return TT_OK;
    }
    // Nothing is cleared in front of the chain: the status word of the header is tagged with the call's epoch, the
    // one counter of the chain (k_merge's tickets) is zeroed by the kernel before it, and every per-tile record has
    // exactly one writer.  A stream capture (whose replays repeat the epoch) clears the header first.
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) { cudaGetLastError(); cap = cudaStreamCaptureStatusActive; }
    // Bulk text (more tiles than a request's job search covers) uses one counter in the first kernel itself, the length
    // of the global list of warp-class pieces: there the header is cleared too.
    const bool big = (((uintptr_t)text & 15) + len + TT_TILE_BYTES - 1) / TT_TILE_BYTES > (size_t)MERGE_SR_MAX_TILES;
    if (doc_off || literals || big || cap != cudaStreamCaptureStatusNone) CK(cudaMemsetAsync(w.hdr, 0, sizeof(TTHeader), st));
    MARK(0);
    PretokParams PP;
    int rc = run_pretok(v, text, len, doc_off, n_docs, st, w, nullptr, PP, literals, true, host_src);
    if (rc != TT_OK) return rc;
    MARK(1);
    const int tile_grid = PP.ntiles < v->sm_count * 8 ? PP.ntiles : v->sm_count * 8;
    const int merge_grid = v->sm_count * MERGE_CTAS_PER_SM;                  // all resident CTA slots: a request's unsettled pieces get a warp each
    PieceParams Q;
    Q.base = PP.base; Q.shift = PP.lo; Q.hi = PP.hi; Q.ntiles = PP.ntiles;
    Q.tile_cnt = w.tile_cnt; Q.tile_first = w.tile_first; Q.tile_last = w.tile_last; Q.tile_q = w.tile_q; Q.tile_long = w.tile_long;
    Q.piece_off16 = w.piece_off16; Q.q = w.q;
    Q.hdr = w.hdr; Q.tab = v->tab; Q.toktab = v->toktab; Q.longtab = v->longtab; Q.litstart = literals ? w.litstart : nullptr; Q.epoch = PP.epoch;
    Q.ext_id = v->d_ext_id; Q.piece_cnt = w.piece_cnt; Q.stage = w.stage; Q.pairbuf = w.pairbuf; Q.tile_tok = w.tile_tok;
    Q.grp_tok = PP.ntiles > MERGE_SR_MAX_TILES ? w.grp_tok : nullptr;   // group totals only where k_scatter's CTAs would otherwise sum thousands of tiles each
    Q.wq = big ? w.wq : nullptr; Q.gq = big ? w.gq : nullptr;
    for (int c = 0; c < TT_SHORT_CLASSES - 1; c++) Q.gq_x[c] = big ? w.gq_x[c] : nullptr; Q.lq = big ? w.lq : nullptr;
    if (big) {                                                               // bulk text: closing pieces and the global lists first
        const int cgrid = (PP.ntiles + CLOSING_THREADS - 1) / CLOSING_THREADS;
        if (ev) k_closing<<<cgrid, CLOSING_THREADS, 0, st>>>(Q);
        else CK(launch_after(k_closing, cgrid, CLOSING_THREADS, st, Q));
    }
    if (ev) { if (big) k_merge_bulk<<<merge_grid, MERGE_THREADS, MERGE_SMEM_BYTES, st>>>(Q); else k_merge<<<merge_grid, MERGE_THREADS, MERGE_SMEM_BYTES, st>>>(Q); }
    else CK(launch_after(big ? k_merge_bulk : k_merge, merge_grid, MERGE_THREADS, st, Q, MERGE_SMEM_BYTES));
    MARK(2);
    ScatterParams S;
    S.shift = PP.lo; S.hi = PP.hi; S.ntiles = PP.ntiles; S.tile_cnt = w.tile_cnt; S.tile_tok = w.tile_tok; S.grp_tok = Q.grp_tok; S.piece_off16 = w.piece_off16;
    S.ids_cap = (unsigned long long)ids_cap; S.piece_cnt = w.piece_cnt; S.stage = w.stage; S.hdr = w.hdr; S.epoch = PP.epoch;
    S.ids_out = ids_out; S.count_out = (long long*)count_out; S.status_out = status_out;
    S.docmask = doc_off ? w.docmask : nullptr; S.doc_off = (const long long*)doc_off; S.n_docs = (int)n_docs;
    S.ids_off_out = (long long*)ids_off_out;
    if (ev) { if (big) k_scatter_bulk<<<tile_grid, BPE_THREADS, 0, st>>>(S); else k_scatter<<<tile_grid, BPE_THREADS, 0, st>>>(S); }
    else CK(launch_after(big ? k_scatter_bulk : k_scatter, tile_grid, BPE_THREADS, st, S));
    MARK(3);
#undef MARK
    CK(cudaGetLastError());
    return TT_OK;
}

extern "C" int tt_encode(const tt_vocab* v, const uint8_t* text, size_t len, void* stream, int32_t* ids_out,
                         size_t ids_cap, int64_t* count_out, int32_t* status_out, void* workspace,
                         size_t workspace_bytes) {
    int rc = check_common(v, text, len, workspace, workspace_bytes, 1);
    if (rc != TT_OK) return rc;
    if (!count_out || !status_out || (len && !ids_out)) return TT_ERR_ARG;
    return encode_impl(v, text, len, nullptr, 1, (cudaStream_t)stream, ids_out, ids_cap, count_out, nullptr, status_out,
                       workspace);
}

extern "C" int tt_vocab_add_literals(tt_vocab* v, const uint8_t* bytes, const uint32_t* off, const int32_t* ids, size_t n) {
    if (!v || v->lit.n != 0 || n == 0 || n > 65535 || !bytes || !off || !ids) return TT_ERR_ARG;
    std::vector<LitEntry> e(n);
    std::unordered_set<std::string> seen;
    u32 maxlen = 0;
    LitTable T{};
    for (size_t i = 0; i < n; i++) {
        if (off[i + 1] <= off[i] || off[i + 1] - off[i] > 255 || ids[i] < 0) return TT_ERR_ARG;
        const u32 len = off[i + 1] - off[i];
        if (!seen.insert(std::string((const char*)bytes + off[i], len)).second) return TT_ERR_ARG;     // the same literal twice
        u32 f4 = 0;
        for (u32 k = 0; k < 4 && k < len; k++) f4 |= (u32)bytes[off[i] + k] << (8 * k);
        e[i].first4 = f4; e[i].off = off[i]; e[i].len = len; e[i].id = ids[i];
        maxlen = maxlen > len ? maxlen : len;
        T.first_byte[bytes[off[i]] >> 5] |= 1u << (bytes[off[i]] & 31);
    }
    std::stable_sort(e.begin(), e.end(), [](const LitEntry& a, const LitEntry& b) { return a.len > b.len; });
    const size_t blob = off[n];
    if (cudaMalloc(&v->d_lit_entries, n * sizeof(LitEntry)) != cudaSuccess || cudaMalloc(&v->d_lit_blob, blob + 16) != cudaSuccess ||
        cudaMemcpy(v->d_lit_entries, e.data(), n * sizeof(LitEntry), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(v->d_lit_blob, bytes, blob, cudaMemcpyHostToDevice) != cudaSuccess) {
        cudaGetLastError(); cudaFree(v->d_lit_entries); cudaFree(v->d_lit_blob); v->d_lit_entries = nullptr; v->d_lit_blob = nullptr;
        return TT_ERR_CUDA;
    }
    T.entries = v->d_lit_entries; T.blob = v->d_lit_blob; T.n = (u32)n; T.maxlen = maxlen;
    // the literals are registered (v->lit) only once every allocation and copy below has succeeded, so that a
    // failed call leaves the vocabulary as it was and may be repeated
    auto undo = [&]() { cudaFree(v->d_lit_entries); cudaFree(v->d_lit_blob); v->d_lit_entries = nullptr; v->d_lit_blob = nullptr; };
    if (v->meta_n) {
        // tt_spans: byte and character length of every literal whose id the merge table does not use itself
        int32_t max_id = (int32_t)v->meta_n - 1;
        for (size_t i = 0; i < n; i++) max_id = ids[i] > max_id ? ids[i] : max_id;
        if (max_id < (1 << 24)) {
            std::vector<uint2> meta((size_t)max_id + 1, make_uint2(0, 0));
            uint2* d_new = nullptr;
            bool ok = cudaMemcpy(meta.data(), v->d_meta, (size_t)v->meta_n * sizeof(uint2), cudaMemcpyDeviceToHost) == cudaSuccess;
            for (size_t i = 0; ok && i < n; i++) {
                if (meta[ids[i]].x != 0) continue;
                u32 chars = 0;
                for (u32 k = off[i]; k < off[i + 1]; k++) chars += (bytes[k] & 0xC0) != 0x80;
                meta[ids[i]] = make_uint2(off[i + 1] - off[i], chars);
            }
            ok = ok && cudaMalloc(&d_new, meta.size() * sizeof(uint2)) == cudaSuccess;
            ok = ok && cudaMemcpy(d_new, meta.data(), meta.size() * sizeof(uint2), cudaMemcpyHostToDevice) == cudaSuccess;
            if (!ok) { cudaGetLastError(); cudaFree(d_new); undo(); return TT_ERR_CUDA; }
            cudaFree(v->d_meta);
            v->d_meta = d_new; v->meta_n = (u32)meta.size();
        }
    }
    v->lit = T;
    return TT_OK;
}

extern "C" int tt_encode_added(const tt_vocab* v, const uint8_t* text, size_t len, void* stream, int32_t* ids_out,
                               size_t ids_cap, int64_t* count_out, int32_t* status_out, void* workspace,
                               size_t workspace_bytes) {
    int rc = check_common(v, text, len, workspace, workspace_bytes, 1);
    if (rc != TT_OK) return rc;
    if (!count_out || !status_out || (len && !ids_out)) return TT_ERR_ARG;
    return encode_impl(v, text, len, nullptr, 1, (cudaStream_t)stream, ids_out, ids_cap, count_out, nullptr, status_out,
                       workspace, nullptr, v->lit.n != 0);
}

extern "C" int tt_encode_batch(const tt_vocab* v, const uint8_t* text, size_t total_len, const int64_t* doc_off,
                               size_t n_docs, void* stream, int32_t* ids_out, size_t ids_cap, int64_t* ids_off_out,
                               int32_t* status_out, void* workspace, size_t workspace_bytes) {
    int rc = check_common(v, text, total_len, workspace, workspace_bytes, n_docs);
    if (rc != TT_OK) return rc;
    if (!doc_off || !ids_off_out || !status_out || (total_len && !ids_out) || n_docs >= (size_t)INT32_MAX) return TT_ERR_ARG;
    return encode_impl(v, text, total_len, doc_off, n_docs, (cudaStream_t)stream, ids_out, ids_cap, nullptr, ids_off_out,
                       status_out, workspace);
}

extern "C" int tt_encode_timed(const tt_vocab* v, const uint8_t* text, size_t len, void* stream, int32_t* ids_out,
                               size_t ids_cap, int64_t* count_out, int32_t* status_out, void* workspace,
                               size_t workspace_bytes, float ms_out[3]) {
    int rc = check_common(v, text, len, workspace, workspace_bytes, 1);
    if (rc != TT_OK) return rc;
    if (!count_out || !status_out || !ms_out || !len || !ids_out) return TT_ERR_ARG;
    cudaEvent_t ev[4];
    for (int i = 0; i < 4; i++) CK(cudaEventCreate(&ev[i]));
    rc = encode_impl(v, text, len, nullptr, 1, (cudaStream_t)stream, ids_out, ids_cap, count_out, nullptr, status_out,
                     workspace, ev);
    if (rc == TT_OK && cudaEventSynchronize(ev[3]) != cudaSuccess) rc = TT_ERR_CUDA;
    for (int i = 0; i < 3 && rc == TT_OK; i++)
        if (cudaEventElapsedTime(&ms_out[i], ev[i], ev[i + 1]) != cudaSuccess) rc = TT_ERR_CUDA;
    for (int i = 0; i < 4; i++) cudaEventDestroy(ev[i]);
    return rc;
}

__global__ void k_finish_pretok(const TTHeader* hdr, unsigned long long epoch, long long* n_pieces_out, int32_t* status_out) {
    const int status = hdr_status(hdr, epoch);
    *status_out = status;
    *n_pieces_out = status ? 0 : (long long)hdr->n_pieces;
}

extern "C" int tt_pretokenize(const tt_vocab* v, const uint8_t* text, size_t len, const int64_t* doc_off, size_t n_docs,
                              void* stream, int32_t* piece_off_out, size_t piece_cap, int64_t* n_pieces_out,
                              int32_t* status_out, void* workspace, size_t workspace_bytes) {
    int rc = check_common(v, text, len, workspace, workspace_bytes, n_docs);
    if (rc != TT_OK) return rc;
    if (!n_pieces_out || !status_out || (len && (!piece_off_out || piece_cap < len + 1))) return TT_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    TTWorkspace w;
    carve(&w, workspace, len, n_docs);
    CK(cudaMemsetAsync(w.hdr, 0, sizeof(TTHeader), st));
    if (len == 0) {
        CK(cudaMemsetAsync(n_pieces_out, 0, sizeof(int64_t), st));
        CK(cudaMemsetAsync(status_out, 0, sizeof(int32_t), st));
        return TT_OK;
    }
    PretokParams PP;
    rc = run_pretok(v, text, len, doc_off, n_docs, st, w, (u32*)piece_off_out, PP);
    if (rc != TT_OK) return rc;
    k_finish_pretok<<<1, 1, 0, st>>>(w.hdr, PP.epoch, (long long*)n_pieces_out, status_out);
    CK(cudaGetLastError());
    return TT_OK;
}

extern "C" size_t tt_spans_workspace_bytes(const tt_vocab* v, size_t ids_cap) {
    (void)v;
    return align_up(sizeof(SpanHeader), 256) + align_up((ids_cap / SPAN_THREADS + 3) * sizeof(uint2), 256);
}

extern "C" int tt_spans(const tt_vocab* v, const int32_t* ids, const int64_t* count, size_t ids_cap, size_t text_len,
                        void* stream, int32_t* byte_off_out, int32_t* char_off_out, int32_t* status_out, void* workspace,
                        size_t workspace_bytes) {
    if (!v || !count || !byte_off_out || !char_off_out || !status_out || !workspace || (ids_cap && !ids)) return TT_ERR_ARG;
    if (v->meta_n == 0 || ids_cap >= (size_t)INT32_MAX || text_len >= (size_t)INT32_MAX) return TT_ERR_ARG;
    if (((uintptr_t)workspace & 255) != 0 || workspace_bytes < tt_spans_workspace_bytes(v, ids_cap)) return TT_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    SpanParams P;
    P.ids = ids; P.count = (const long long*)count; P.ids_cap = ids_cap; P.text_len = text_len;
    P.meta = v->d_meta; P.meta_n = v->meta_n;
    P.hdr = (SpanHeader*)workspace;
    P.blk = (uint2*)((char*)workspace + align_up(sizeof(SpanHeader), 256));
    P.byte_off = byte_off_out; P.char_off = char_off_out; P.status_out = status_out;
    CK(cudaMemsetAsync(P.hdr, 0, sizeof(SpanHeader), st));
    size_t want = (ids_cap + SPAN_THREADS - 1) / SPAN_THREADS;
    if (want < 1) want = 1;
    const int grid = (int)(want > (size_t)v->sm_count * 2 ? (size_t)v->sm_count * 2 : want);
    k_span_sums<<<grid, SPAN_THREADS, 0, st>>>(P);
    k_span_write<<<grid, SPAN_THREADS, 0, st>>>(P);
    CK(cudaGetLastError());
    return TT_OK;
}

// Is p page-locked host memory?  dev_view (optional) receives the pointer a kernel may use to reach it.
static bool host_pointer_is_pinned(const void* p, void** dev_view) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) { cudaGetLastError(); return false; }
    if (a.type != cudaMemoryTypeHost) return false;
    if (dev_view) *dev_view = a.devicePointer;
    return true;
}

extern "C" int tt_encode_host(tt_vocab* v, const uint8_t* text, size_t len, int32_t* ids_out, size_t ids_cap,
                              int64_t* count_out) {
    if (!v || !count_out || (len && (!text || !ids_out))) return TT_ERR_ARG;
    if (len >= (size_t)INT32_MAX - 64) return TT_ERR_ARG;
    *count_out = 0;
    if (!v->host_stream) CK(cudaStreamCreateWithFlags(&v->host_stream, cudaStreamNonBlocking));
    if (len + 1 > v->host_cap) {
        cudaFree(v->d_text); cudaFree(v->d_ids); cudaFree(v->d_ws);
        if (v->h_text) cudaFreeHost(v->h_text);
        if (v->h_ids) cudaFreeHost(v->h_ids);
        v->d_text = nullptr; v->d_ids = nullptr; v->d_ws = nullptr; v->h_text = nullptr; v->h_ids = nullptr; v->host_cap = 0;
        const size_t cap = align_up(len + 1 + len / 4, 4096);
        v->ws_cap = tt_workspace_bytes(v, cap, 1);
        CK(cudaMalloc(&v->d_text, cap + 64));
        CK(cudaMalloc(&v->d_ids, cap * sizeof(int32_t)));
        CK(cudaMalloc(&v->d_ws, v->ws_cap));
        CK(cudaMallocHost(&v->h_text, cap + 64));
        CK(cudaMallocHost(&v->h_ids, cap * sizeof(int32_t)));
        if (!v->d_count) CK(cudaMalloc(&v->d_count, sizeof(long long)));
        if (!v->d_status) CK(cudaMalloc(&v->d_status, sizeof(int32_t)));
        if (!v->h_scalars) CK(cudaMallocHost(&v->h_scalars, 2 * sizeof(long long)));
        v->host_cap = cap;
    }
    cudaStream_t st = v->host_stream;
    // Pinned (page-locked) caller buffers take no staging: the text is copied by DMA straight from the caller's
    // buffer, and the scatter kernel writes the ids through the mapped pointer straight into the caller's
    // buffer, so no device-to-host copy follows.  Pageable buffers go through the handle's pinned staging.
    int32_t* ids_dev_view = nullptr;
    const uint8_t* text_dev_view = nullptr;
    const bool in_pinned = len && host_pointer_is_pinned(text, (void**)&text_dev_view) && text_dev_view != nullptr;
    const bool out_pinned = len && host_pointer_is_pinned(ids_out, (void**)&ids_dev_view) && ids_dev_view != nullptr;
    // Pinned text is not copied in front of the chain: the first kernel reads it through the mapped pointer, tile by
    // tile, and leaves the device copy that the later kernels need -- the transfer runs under the kernel's own work.
    const uint8_t* d_text = in_pinned ? v->d_text + ((uintptr_t)text_dev_view & 15) : v->d_text;
    if (!in_pinned) {
        // pageable text is staged in slices, so that the DMA of one slice runs while the next is being staged
        const size_t slice = 256u << 10;
        for (size_t o = 0; o < len; o += slice) {
            const size_t n = len - o < slice ? len - o : slice;
            memcpy(v->h_text + o, text + o, n);
            CK(cudaMemcpyAsync(v->d_text + o, v->h_text + o, n, cudaMemcpyHostToDevice, st));
        }
    }
    // count and status are written by the kernel into mapped pinned scalars of the handle
    long long* count_dev = nullptr; int32_t* status_dev = nullptr;
    {
        if (!v->h_scalars_dev) {                                  // looked up once: the buffer lives as long as the handle
            void* p = nullptr;
            if (!host_pointer_is_pinned(v->h_scalars, &p) || !p) return TT_ERR_CUDA;
            v->h_scalars_dev = (long long*)p;
        }
        count_dev = v->h_scalars_dev; status_dev = (int32_t*)(v->h_scalars_dev + 1);
    }
    v->h_scalars[0] = 0; v->h_scalars[1] = 0;
    if (v->ws_cap < tt_workspace_bytes(v, len, 1)) return TT_ERR_ARG;
    int rc = encode_impl(v, d_text, len, nullptr, 1, st, out_pinned ? ids_dev_view : v->d_ids, out_pinned ? ids_cap : v->host_cap,
                         (int64_t*)count_dev, nullptr, status_dev, v->d_ws, nullptr, false, in_pinned ? text_dev_view : nullptr);
    if (rc != TT_OK) return rc;
    CK(cudaStreamSynchronize(st));
    const int status = (int)(v->h_scalars[1] & 0xFFFFFFFF);
    if (status != TT_OK) return status;
    const long long n = v->h_scalars[0];
    if ((size_t)n > ids_cap) return TT_ERR_CAPACITY;
    if (!out_pinned && n > 0) {
        // the ids come back in up to eight slices: while one is copied out of the staging buffer the DMA brings the next
        const size_t total = (size_t)n * sizeof(int32_t);
        size_t nsl = (total + (256u << 10) - 1) / (256u << 10);
        if (nsl > 8) nsl = 8;
        const size_t per = align_up((total + nsl - 1) / nsl, 4096);
        for (size_t k = 0; k < nsl; k++) {
            if (!v->slice_ev[k]) CK(cudaEventCreateWithFlags(&v->slice_ev[k], cudaEventDisableTiming));
            const size_t o = k * per, nb = o >= total ? 0 : (total - o < per ? total - o : per);
            if (nb) CK(cudaMemcpyAsync((char*)v->h_ids + o, (const char*)v->d_ids + o, nb, cudaMemcpyDeviceToHost, st));
            CK(cudaEventRecord(v->slice_ev[k], st));
        }
        for (size_t k = 0; k < nsl; k++) {
            CK(cudaEventSynchronize(v->slice_ev[k]));
            const size_t o = k * per, nb = o >= total ? 0 : (total - o < per ? total - o : per);
            if (nb) memcpy((char*)ids_out + o, (const char*)v->h_ids + o, nb);
        }
    }
    *count_out = n;
    return TT_OK;
}

// ---- entry point that needs no caller scratch and allocates nothing ---------------------------------
// The scratch of the kernel chain lives in a fixed device array that is part of the library image, so
// every GPU that loads the library carries it until the process exits.
#define TT_STATIC_SCRATCH_BYTES ((size_t)TT_STATIC_MAX_LEN * 28u + 65536u)
static __device__ __align__(256) unsigned char tt_static_scratch[TT_STATIC_SCRATCH_BYTES];

// Host code may not use the array's name as an address (it names a host-side shadow); the device
// address is looked up once per device and remembered.
static void* g_static_scratch_ptr[64];
static std::mutex g_static_scratch_mutex;

extern "C" int tt_encode_static(const tt_vocab* v, const uint8_t* text, size_t len, void* stream, int32_t* ids_out,
                                size_t ids_cap, int64_t* count_out, int32_t* status_out) {
    if (!v || !count_out || !status_out || (len && (!text || !ids_out))) return TT_ERR_ARG;
    if (len > TT_STATIC_MAX_LEN) return TT_ERR_TOO_LARGE;
    if (carve(nullptr, nullptr, len, 1) > TT_STATIC_SCRATCH_BYTES) return TT_ERR_TOO_LARGE;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return TT_ERR_CUDA; }
    if (dev < 0 || dev >= 64) return TT_ERR_ARG;
    void* scratch = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
        if (!g_static_scratch_ptr[dev]) {                        // first call on this device: set-up
            void* p = nullptr;
            if (cudaGetSymbolAddress(&p, tt_static_scratch) != cudaSuccess || !p) { cudaGetLastError(); return TT_ERR_CUDA; }
            g_static_scratch_ptr[dev] = p;
        }
        scratch = g_static_scratch_ptr[dev];
    }
    // Nothing of the previous call's contents matters: the chain's first kernel zeroes the header's work
    // counters, the status word is tagged with this call's epoch (an older tag reads as "no error"; encode_impl
    // clears the header with a memset only under stream capture), and every other scratch array is written
    // before it is read.
    return encode_impl(v, text, len, nullptr, 1, (cudaStream_t)stream, ids_out, ids_cap, count_out, nullptr, status_out,
                       scratch);
}

// ---- sessions: incremental repair on append (paper Sec. 3.3) ------------------------------------------
struct tt_session {
    const tt_vocab* v = nullptr;
    size_t cap = 0;                       // bytes of text the session can hold
    size_t len = 0;                       // bytes stored
    uint32_t window_chars = 512;
    std::vector<u8> h_tail;               // host copy of the END of the stored text only: the window starts are found here
    size_t tail_base = 0;                 // (text offset of h_tail[0]; enough for the widest window, see session_keep_tail)
    u8* d_text = nullptr;
    int32_t *d_ids = nullptr, *d_off = nullptr;                 // cached records; d_off[ntok] = len
    int32_t *d_fids = nullptr, *d_foff = nullptr, *d_fchar = nullptr;   // fresh records / scratch of the span export
    u8* d_eq = nullptr;
    long long *d_ntok = nullptr, *d_fcount = nullptr;
    int32_t *d_fstatus = nullptr, *d_sstatus = nullptr;
    RepairDecision* d_dec = nullptr;
    struct Host { RepairDecision dec; long long ntok; int32_t fstatus, sstatus; }* h = nullptr;   // pinned
    void *d_ws = nullptr, *d_sws = nullptr;
    size_t ws_bytes = 0, sws_bytes = 0;
};

extern "C" void tt_session_free(tt_session* s) {
    if (!s) return;
    cudaFree(s->d_text); cudaFree(s->d_ids); cudaFree(s->d_off); cudaFree(s->d_fids); cudaFree(s->d_foff); cudaFree(s->d_fchar);
    cudaFree(s->d_eq); cudaFree(s->d_ntok); cudaFree(s->d_fcount); cudaFree(s->d_fstatus); cudaFree(s->d_sstatus);
    cudaFree(s->d_dec); cudaFree(s->d_ws); cudaFree(s->d_sws);
    if (s->h) cudaFreeHost(s->h);
    delete s;
}

extern "C" int tt_session_create(const tt_vocab* v, size_t max_bytes, tt_session** out) {
    if (out) *out = nullptr;
    if (!v || !out || max_bytes == 0 || max_bytes >= (size_t)INT32_MAX - 64 || v->meta_n == 0) return TT_ERR_ARG;
    tt_session* s = new (std::nothrow) tt_session();
    if (!s) return TT_ERR_CUDA;
    s->v = v; s->cap = max_bytes;
    s->ws_bytes = tt_workspace_bytes(v, max_bytes, 1);
    s->sws_bytes = tt_spans_workspace_bytes(v, max_bytes);
    const size_t n1 = max_bytes + 1;
    bool ok = cudaMalloc(&s->d_text, max_bytes + 64) == cudaSuccess && cudaMalloc(&s->d_ids, n1 * 4) == cudaSuccess &&
              cudaMalloc(&s->d_off, n1 * 4) == cudaSuccess && cudaMalloc(&s->d_fids, n1 * 4) == cudaSuccess &&
              cudaMalloc(&s->d_foff, n1 * 4) == cudaSuccess && cudaMalloc(&s->d_fchar, n1 * 4) == cudaSuccess &&
              cudaMalloc(&s->d_eq, n1) == cudaSuccess && cudaMalloc(&s->d_ntok, 8) == cudaSuccess &&
              cudaMalloc(&s->d_fcount, 8) == cudaSuccess && cudaMalloc(&s->d_fstatus, 4) == cudaSuccess &&
              cudaMalloc(&s->d_sstatus, 4) == cudaSuccess && cudaMalloc(&s->d_dec, sizeof(RepairDecision)) == cudaSuccess &&
              cudaMalloc(&s->d_ws, s->ws_bytes) == cudaSuccess && cudaMalloc(&s->d_sws, s->sws_bytes) == cudaSuccess &&
              cudaMallocHost(&s->h, sizeof(tt_session::Host)) == cudaSuccess;
    ok = ok && cudaMemset(s->d_ntok, 0, 8) == cudaSuccess && cudaMemset(s->d_off, 0, 4) == cudaSuccess;
    if (!ok) { cudaGetLastError(); tt_session_free(s); return TT_ERR_CUDA; }
    *out = s;
    return TT_OK;
}

extern "C" int tt_session_set_window(tt_session* s, uint32_t window_chars) {
    if (!s || window_chars == 0 || window_chars > (1u << 24)) return TT_ERR_ARG;
    s->window_chars = window_chars;
    return TT_OK;
}

extern "C" int tt_session_view(const tt_session* s, const int32_t** ids_dev, const int32_t** off_dev,
                               const int64_t** count_dev, size_t* len_bytes) {
    if (!s) return TT_ERR_ARG;
    if (ids_dev) *ids_dev = s->d_ids;
    if (off_dev) *off_dev = s->d_off;
    if (count_dev) *count_dev = (const int64_t*)s->d_ntok;
    if (len_bytes) *len_bytes = s->len;
    return TT_OK;
}

// Tokenizes text[from, new_len) into (ids, off, count) with offsets relative to `from`.
static int session_tokenize(tt_session* s, size_t from, size_t new_len, cudaStream_t st, int32_t* ids, int32_t* off, long long* count) {
    const size_t n = new_len - from;
    int rc = encode_impl(s->v, s->d_text + from, n, nullptr, 1, st, ids, s->cap, (int64_t*)count, nullptr, s->d_fstatus, s->d_ws);
    if (rc != TT_OK) return rc;
    return tt_spans(s->v, ids, (const int64_t*)count, s->cap, n, st, off, s->d_fchar, s->d_sstatus, s->d_sws, s->sws_bytes);
}

// The host keeps the last bytes of the stored text, as many as the widest window of the protocol can span (five
// doublings of the window, four bytes a character): an append costs a copy of that tail at most, whatever the
// session holds.
static void session_keep_tail(tt_session* s, const uint8_t* text, size_t len) {
    const size_t keep = (size_t)s->window_chars * 32 * 4 + 64;
    s->h_tail.insert(s->h_tail.end(), text, text + len);
    if (s->h_tail.size() > 2 * keep) {
        const size_t drop = s->h_tail.size() - keep;
        s->h_tail.erase(s->h_tail.begin(), s->h_tail.begin() + (ptrdiff_t)drop);
        s->tail_base += drop;
    }
}

extern "C" int tt_session_append(tt_session* s, const uint8_t* text, size_t len, void* stream, tt_append_info* info) {
    if (!s || (len && !text)) return TT_ERR_ARG;
    if (len > s->cap - s->len) return TT_ERR_TOO_LARGE;
    cudaStream_t st = (cudaStream_t)stream;
    tt_append_info local; memset(&local, 0, sizeof(local));
    const size_t old_len = s->len, new_len = old_len + len;
    // (an error return waits for the stream first: the copy from the caller's buffer may still be in flight)
    auto fail = [&](int code) { cudaStreamSynchronize(st); cudaGetLastError(); if (info) { local.status = code; *info = local; } return code; };
    if (len) { if (cudaMemcpyAsync(s->d_text + old_len, text, len, cudaMemcpyHostToDevice, st) != cudaSuccess) { cudaGetLastError(); return fail(TT_ERR_CUDA); } }
    if (new_len == 0) { if (info) *info = local; return TT_OK; }
    const u8* ht = s->h_tail.data() - s->tail_base;          // ht[i] = byte i of the stored text, for i >= tail_base
    uint64_t w = s->window_chars;
    for (int attempt = 0; attempt <= 5 && old_len > 0; attempt++, w *= 2) {
        // byte offset of the character that lies w characters before the end of the stored text
        size_t ws = old_len; uint64_t left = w;
        while (ws > s->tail_base && left > 0) { ws--; while (ws > s->tail_base && (ht[ws] & 0xC0) == 0x80) ws--; left--; }
        if (left > 0 || ws == s->tail_base) ws = 0;           // the window reaches the start of the text (or beyond what the host kept: more work, same ids)
        local.attempts = attempt + 1;
        if (ws == 0) break;                                   // the window is the whole text
        int rc = session_tokenize(s, ws, new_len, st, s->d_fids, s->d_foff, s->d_fcount);
        if (rc != TT_OK) return fail(rc);
        RepairParams P;
        P.ids = s->d_ids; P.off = s->d_off; P.ntok = s->d_ntok;
        P.fids = s->d_fids; P.foff = s->d_foff; P.fchar = s->d_fchar; P.fcount = s->d_fcount;
        P.fstatus = s->d_fstatus; P.sstatus = s->d_sstatus; P.text = s->d_text;
        P.ws = (long long)ws; P.old_len = (long long)old_len; P.new_len = (long long)new_len;
        P.cls = s->v->d_cls; P.cls_bytes = s->v->cls_bytes; P.max_tok_chars = (int)s->v->max_token_chars;
        P.eq = s->d_eq; P.dec = s->d_dec;
        k_repair_decide<<<1, 256, 0, st>>>(P);
        const size_t fresh_max = new_len - ws;
        const int grid = (int)((fresh_max + 255) / 256 < (size_t)s->v->sm_count * 4 ? (fresh_max + 255) / 256 : (size_t)s->v->sm_count * 4);
        k_repair_apply<<<grid, 256, 0, st>>>(P);
        if (cudaMemcpyAsync(&s->h->dec, s->d_dec, sizeof(RepairDecision), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
            cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return fail(TT_ERR_CUDA); }
        const RepairDecision d = s->h->dec;
        if (d.status != TT_OK) return fail(d.status);          // e.g. the appended text is not valid UTF-8: nothing changed
        if (d.accept) {
            s->len = new_len; session_keep_tail(s, text, len);
            local.window_chars = (int64_t)w; local.window_start = (int64_t)ws; local.run_tokens = d.j1 - d.j0;
            local.splice_byte = d.splice_byte; local.n_tokens = d.new_ntok; local.status = TT_OK;
            if (info) *info = local;
            return TT_OK;
        }
    }
    if (local.attempts == 0) local.attempts = 1;
    // full tokenization straight into the session's records (into the fresh buffers first, so that an error
    // leaves the session as it was)
    int rc = session_tokenize(s, 0, new_len, st, s->d_fids, s->d_foff, s->d_fcount);
    if (rc != TT_OK) return fail(rc);
    if (cudaMemcpyAsync(&s->h->ntok, s->d_fcount, 8, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(&s->h->fstatus, s->d_fstatus, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaMemcpyAsync(&s->h->sstatus, s->d_sstatus, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return fail(TT_ERR_CUDA); }
    if (s->h->fstatus != TT_OK) return fail(s->h->fstatus);
    if (s->h->sstatus != TT_OK) return fail(s->h->sstatus);
    const size_t nt = (size_t)s->h->ntok;
    if (cudaMemcpyAsync(s->d_ids, s->d_fids, nt * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(s->d_off, s->d_foff, (nt + 1) * 4, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(s->d_ntok, s->d_fcount, 8, cudaMemcpyDeviceToDevice, st) != cudaSuccess ||
        cudaStreamSynchronize(st) != cudaSuccess) { cudaGetLastError(); return fail(TT_ERR_CUDA); }
    s->len = new_len; session_keep_tail(s, text, len);
    local.window_chars = 0; local.window_start = 0; local.run_tokens = 0; local.splice_byte = 0;
    local.n_tokens = (int64_t)nt; local.status = TT_OK;
    if (info) *info = local;
    return TT_OK;
}

extern "C" int tt_session_copy(const tt_session* s, int32_t* ids_out, size_t ids_cap, int32_t* off_out,
                               int64_t* count_out, void* stream) {
    if (!s || !count_out) return TT_ERR_ARG;
    cudaStream_t st = (cudaStream_t)stream;
    // the count is known on the host only as an upper bound (one token per byte); copy by that bound
    const size_t n = s->len < ids_cap ? s->len : ids_cap;
    if (ids_out && n) CK(cudaMemcpyAsync(ids_out, s->d_ids, n * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    if (off_out) CK(cudaMemcpyAsync(off_out, s->d_off, (n + 1) * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    CK(cudaMemcpyAsync(count_out, s->d_ntok, sizeof(int64_t), cudaMemcpyDeviceToDevice, st));
    return TT_OK;
}

// ---- shadow verification (paper Sec. 4.4) ---------------------------------------------------------------
// Host-only: a background thread re-tokenizes a sample of the emitted sequences with a reference engine
// supplied by the caller and compares ids exactly; mismatches are kept with a content hash; when the queue
// is full samples are dropped and counted.
#include <condition_variable>
#include <deque>
#include <thread>

struct tt_verifier {
    tt_reference_fn ref = nullptr; void* user = nullptr;
    double rate = 1.0; size_t queue_cap = 64; uint64_t seed = 0;
    struct Item { std::vector<u8> text; std::vector<int32_t> ids; };
    std::deque<Item> queue;
    std::mutex mu; std::condition_variable cv_work, cv_idle;
    bool stop = false, busy = false;
    tt_verifier_stats st{};
    struct Bad { uint64_t hash; uint64_t len; int64_t first_diff; };
    std::vector<Bad> quarantine;
    std::thread worker;
};

static uint64_t verifier_hash(const u8* p, size_t n) {          // FNV-1a, 64 bit
    uint64_t h = 0xCBF29CE484222325ull;
    for (size_t i = 0; i < n; i++) { h ^= p[i]; h *= 0x100000001B3ull; }
    return h;
}
static uint64_t verifier_mix(uint64_t x) {                       // splitmix64 finaliser: the sampling decision of submission x
    x += 0x9E3779B97F4A7C15ull; x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull; x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
    return x ^ (x >> 31);
}

static void verifier_loop(tt_verifier* q) {
    std::vector<int32_t> out;
    for (;;) {
        tt_verifier::Item it;
        {
            std::unique_lock<std::mutex> lk(q->mu);
            q->busy = false;
            if (q->queue.empty()) q->cv_idle.notify_all();
            q->cv_work.wait(lk, [&] { return q->stop || !q->queue.empty(); });
            if (q->queue.empty()) return;                        // stop requested and nothing left
            it = std::move(q->queue.front()); q->queue.pop_front();
            q->busy = true;
        }
        out.assign(it.text.size() + 1, 0);
        int64_t n = 0;
        const int rc = q->ref(q->user, it.text.data(), it.text.size(), out.data(), out.size(), &n);
        int64_t diff = -1;
        if (rc != 0 || n < 0 || (size_t)n != it.ids.size()) diff = rc != 0 ? -2 : (int64_t)std::min<size_t>((size_t)(n < 0 ? 0 : n), it.ids.size());
        if (diff == -1) for (size_t i = 0; i < it.ids.size(); i++) if (out[i] != it.ids[i]) { diff = (int64_t)i; break; }
        std::lock_guard<std::mutex> lk(q->mu);
        q->st.checked++;
        if (diff != -1) {
            q->st.mismatches++;
            if (q->quarantine.size() < 4096) q->quarantine.push_back({verifier_hash(it.text.data(), it.text.size()), it.text.size(), diff});
        }
    }
}

extern "C" int tt_verifier_create(tt_reference_fn reference, void* user, double sample_rate, size_t queue_cap, uint64_t seed,
                                  tt_verifier** out) {
    if (out) *out = nullptr;
    if (!reference || !out || !(sample_rate >= 0.0 && sample_rate <= 1.0) || queue_cap == 0) return TT_ERR_ARG;
    tt_verifier* q = new (std::nothrow) tt_verifier();
    if (!q) return TT_ERR_CUDA;
    q->ref = reference; q->user = user; q->rate = sample_rate; q->queue_cap = queue_cap; q->seed = seed;
    q->worker = std::thread(verifier_loop, q);
    *out = q;
    return TT_OK;
}

extern "C" int tt_verifier_submit(tt_verifier* q, const uint8_t* text, size_t len, const int32_t* ids, size_t n_ids) {
    if (!q || (len && !text) || (n_ids && !ids)) return -1;
    std::unique_lock<std::mutex> lk(q->mu);
    const uint64_t k = q->st.submitted++;
    const double u = (double)(verifier_mix(q->seed + k) >> 11) * (1.0 / 9007199254740992.0);
    if (!(u < q->rate)) return 0;
    q->st.sampled++;
    if (q->queue.size() >= q->queue_cap) { q->st.dropped++; return 2; }    // behind: drop, visibly
    lk.unlock();
    tt_verifier::Item it;
    it.text.assign(text, text + len); it.ids.assign(ids, ids + n_ids);
    lk.lock();
    if (q->queue.size() >= q->queue_cap) { q->st.dropped++; return 2; }
    q->queue.push_back(std::move(it));
    q->cv_work.notify_one();
    return 1;
}

extern "C" void tt_verifier_drain(tt_verifier* q) {
    if (!q) return;
    std::unique_lock<std::mutex> lk(q->mu);
    q->cv_idle.wait(lk, [&] { return q->queue.empty() && !q->busy; });
}

extern "C" void tt_verifier_get_stats(tt_verifier* q, tt_verifier_stats* out) {
    if (!q || !out) return;
    std::lock_guard<std::mutex> lk(q->mu);
    *out = q->st;
}

extern "C" int tt_verifier_quarantined(tt_verifier* q, size_t index, uint64_t* content_hash, uint64_t* len, int64_t* first_diff) {
    if (!q) return TT_ERR_ARG;
    std::lock_guard<std::mutex> lk(q->mu);
    if (index >= q->quarantine.size()) return TT_ERR_ARG;
    if (content_hash) *content_hash = q->quarantine[index].hash;
    if (len) *len = q->quarantine[index].len;
    if (first_diff) *first_diff = q->quarantine[index].first_diff;
    return TT_OK;
}

extern "C" void tt_verifier_free(tt_verifier* q) {
    if (!q) return;
    { std::lock_guard<std::mutex> lk(q->mu); q->stop = true; }
    q->cv_work.notify_all();
    if (q->worker.joinable()) q->worker.join();
    delete q;
}

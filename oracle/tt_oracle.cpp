/*
 * CPU ORACLE for exact full-request tokenization  --  TEST INFRASTRUCTURE ONLY.
 *
 * A plain, sequential, deliberately slow statement of what the GPU path must compute:
 * GPT-family regex pre-tokenization (paper Sec. 4.1: a leftmost-first alternation regex,
 * each match beginning where the previous one ended) followed by byte-level BPE applied to
 * every piece independently (paper Sec. 4.2).  Only the tests, the smoke check and the
 * bench's cpu_baseline / reference legs may call into this file.  It shares no code, header,
 * table or constant with the CUDA path.
 *
 * The paper prints neither the regex nor the merge procedure; the two patterns below are the
 * benchmark's "cl100k-style" (pattern 0) and "o200k-style" (pattern 1) alternations, written
 * here as a sequential matcher that tries the alternatives in order at the current position
 * exactly as a backtracking engine would, without using a regex engine.  The tests pin it
 * against a backtracking regex engine on exhaustive small alphabets.
 *
 * Pins (tests/test_oracle_*.py): regex-engine equality, worked examples (tests/golden),
 * pieces-concatenate-to-input, decode(encode(x)) == x, brute-force BPE on tiny tables,
 * equality with an independent byte-pair encoder library fed the same ranks.
 */
#include <cstdint>
#include <cstddef>
#include <cstring>
#include <vector>
#include <string>
#include <unordered_map>
#include <queue>
#include <algorithm>
#include <thread>

namespace {

/* character classes (paper Sec. 4.1: letter, number, whitespace, other; pattern 1 also
 * distinguishes letter case and marks).  The table itself is supplied by the Python side
 * from the interpreter's Unicode database. */
enum : uint8_t { K_O = 0, K_LL = 1, K_LU = 2, K_LB = 3, K_N = 4, K_W = 5, K_M = 6 };

const uint8_t *g_cls = nullptr;   /* 0x110000 entries */

struct Text {
    std::vector<uint32_t> cp;     /* code points */
    std::vector<int64_t> off;     /* byte offset of each code point, plus the total at the end */
};

/* Strict UTF-8 decoding: no overlong forms, no surrogates, nothing above U+10FFFF, no truncation. */
bool decode_utf8(const uint8_t *s, size_t len, Text &t) {
    t.cp.clear(); t.off.clear();
    size_t i = 0;
    while (i < len) {
        uint8_t b = s[i];
        uint32_t c; int n;
        if (b < 0x80) { c = b; n = 1; }
        else if (b >= 0xC2 && b <= 0xDF) { c = b & 0x1F; n = 2; }
        else if (b >= 0xE0 && b <= 0xEF) { c = b & 0x0F; n = 3; }
        else if (b >= 0xF0 && b <= 0xF4) { c = b & 0x07; n = 4; }
        else return false;
        if (i + n > len) return false;
        for (int k = 1; k < n; k++) {
            uint8_t x = s[i + k];
            if ((x & 0xC0) != 0x80) return false;
            c = (c << 6) | (x & 0x3F);
        }
        if (n == 3 && (c < 0x800 || (c >= 0xD800 && c <= 0xDFFF))) return false;
        if (n == 4 && (c < 0x10000 || c > 0x10FFFF)) return false;
        t.cp.push_back(c); t.off.push_back((int64_t)i);
        i += n;
    }
    t.off.push_back((int64_t)len);
    return true;
}

struct Matcher {
    const std::vector<uint32_t> &s;
    size_t n;
    explicit Matcher(const Text &t) : s(t.cp), n(t.cp.size()) {}

    uint8_t k(size_t i) const { return g_cls[s[i]]; }
    bool isNL(size_t i) const { return s[i] == '\n' || s[i] == '\r'; }
    bool isLetter(size_t i) const { uint8_t c = k(i); return c == K_LL || c == K_LU || c == K_LB; }
    bool isN(size_t i) const { return k(i) == K_N; }
    bool isW(size_t i) const { return k(i) == K_W; }
    /* [^\s\p{L}\p{N}] : everything that is not whitespace, letter or number (marks included) */
    bool isOther(size_t i) const { uint8_t c = k(i); return c == K_O || c == K_M; }
    /* [^\r\n\p{L}\p{N}] : the optional one-character prefix of a word piece */
    bool isPrefix(size_t i) const { return !isNL(i) && !isLetter(i) && !isN(i); }

    /* '(?:[sStTmMdD]|[rR][eE]|[vV][eE]|[lL][lL])  -- ASCII letters only, explicit classes */
    size_t contraction(size_t p) const {
        if (p >= n || s[p] != '\'') return 0;
        if (p + 1 < n) {
            uint32_t a = s[p + 1];
            if (a == 's' || a == 'S' || a == 't' || a == 'T' || a == 'm' || a == 'M' || a == 'd' || a == 'D') return 2;
        }
        if (p + 2 < n) {
            uint32_t a = s[p + 1], b = s[p + 2];
            if ((a == 'r' || a == 'R') && (b == 'e' || b == 'E')) return 3;
            if ((a == 'v' || a == 'V') && (b == 'e' || b == 'E')) return 3;
            if ((a == 'l' || a == 'L') && (b == 'l' || b == 'L')) return 3;
        }
        return 0;
    }

    /* alternatives shared by both patterns --------------------------------------------- */
    /* \p{N}{1,3}, or a single \p{N} in the single-digit variant (pattern 2) */
    size_t maxDigits = 3;
    size_t altNumber(size_t p) const {
        size_t e = p;
        while (e < n && e < p + maxDigits && isN(e)) e++;
        return e - p;
    }
    /*  ?[^\s\p{L}\p{N}]+[\r\n]*   (pattern 1: trailing class is [\r\n/]) */
    size_t altPunct(size_t p, bool slashTail) const {
        size_t q;
        if (s[p] == ' ' && p + 1 < n && isOther(p + 1)) q = p + 1;
        else if (isOther(p)) q = p;
        else return 0;
        while (q < n && isOther(q)) q++;
        while (q < n && (isNL(q) || (slashTail && s[q] == '/'))) q++;
        return q - p;
    }
    /* \s*[\r\n]+  |  \s+(?!\S)  |  \s+   tried in this order */
    size_t altSpace(size_t p) const {
        if (!isW(p)) return 0;
        size_t e = p;
        while (e < n && isW(e)) e++;
        /* \s*[\r\n]+ : greedy \s* backs off to the last CR/LF of the whitespace run */
        size_t j = n;
        for (size_t x = p; x < e; x++) if (isNL(x)) j = x;
        if (j != n) return j + 1 - p;
        /* \s+(?!\S) : whole run at end of text; otherwise all but the last whitespace char */
        if (e == n) return e - p;
        if (e - p >= 2) return e - 1 - p;
        /* \s+ */
        return e - p;
    }

    /* pattern 0 ------------------------------------------------------------------------- */
    size_t match0(size_t p) const {
        size_t m = contraction(p);
        if (m) return m;
        /* [^\r\n\p{L}\p{N}]?\p{L}+ */
        if (isPrefix(p) && p + 1 < n && isLetter(p + 1)) {
            size_t e = p + 1; while (e < n && isLetter(e)) e++; return e - p;
        }
        if (isLetter(p)) { size_t e = p; while (e < n && isLetter(e)) e++; return e - p; }
        if ((m = altNumber(p))) return m;
        if ((m = altPunct(p, false))) return m;
        return altSpace(p);
    }

    /* pattern 1 ------------------------------------------------------------------------- */
    /* U = [\p{Lu}\p{Lt}\p{Lm}\p{Lo}\p{M}],  Lw = [\p{Ll}\p{Lm}\p{Lo}\p{M}] */
    bool isWord(size_t i) const { return i < n && (isLetter(i) || k(i) == K_M); }
    bool isU(size_t i) const { uint8_t c = k(i); return c == K_LU || c == K_LB || c == K_M; }
    bool isLw(size_t i) const { uint8_t c = k(i); return c == K_LL || c == K_LB || c == K_M; }
    /* U* Lw+ from q: returns the end, or q if it fails.  Greedy U* then backtracking into Lw+. */
    size_t bodyLower(size_t q) const {
        if (!isWord(q)) return q;
        size_t t = q;
        while (isWord(t) && isU(t)) t++;
        if (isWord(t) && isLw(t)) { size_t v = t; while (isWord(v) && isLw(v)) v++; return v; }
        /* U* swallowed everything it could and nothing of Lw follows: give characters back until
         * the last one kept by Lw+ is in both classes; Lw+ then re-extends greedily to that point. */
        for (size_t x = t; x > q; x--) if (isLw(x - 1)) return x;
        return q;
    }
    /* U+ Lw* from q */
    size_t bodyUpper(size_t q) const {
        if (!isWord(q) || !isU(q)) return q;
        size_t t = q;
        while (isWord(t) && isU(t)) t++;
        while (isWord(t) && isLw(t)) t++;
        return t;
    }
    size_t match1(size_t p) const {
        size_t end = 0; bool ok = false;
        for (int alt = 0; alt < 2 && !ok; alt++) {
            /* optional prefix is greedy: try with it first, then without */
            if (isPrefix(p) && p + 1 < n) {
                size_t v = alt == 0 ? bodyLower(p + 1) : bodyUpper(p + 1);
                if (v > p + 1) { end = v; ok = true; break; }
            }
            size_t v = alt == 0 ? bodyLower(p) : bodyUpper(p);
            if (v > p) { end = v; ok = true; }
        }
        if (ok) return end + contraction(end) - p;
        size_t m;
        if ((m = altNumber(p))) return m;
        if ((m = altPunct(p, true))) return m;
        return altSpace(p);
    }
};

/* piece starts as code-point indices */
void pretok_plain(const Text &t, int pattern, std::vector<size_t> &starts) {
    Matcher M(t);
    if (pattern == 2) M.maxDigits = 1;        /* pattern 2 = pattern 0 with \p{N} in place of \p{N}{1,3} */
    size_t p = 0;
    starts.clear();
    while (p < M.n) {
        starts.push_back(p);
        size_t m = pattern == 1 ? M.match1(p) : M.match0(p);
        if (m == 0) m = 1;   /* cannot happen: every position matches some alternative */
        p += m;
    }
}

/* Pattern 3: three splitters in sequence (paper Sec. 4.1: each splitter re-splits every piece of the stage
 * before it, and the spans a splitter does not match survive as pieces of their own).
 *   A  \p{N}{1,3}        matches isolated
 *   B  [\p{Lm}\p{Lo}]+   (caseless letters: CJK and the like) matches isolated
 *   C  pattern 0 applied to every piece of A.B as a text of its own
 * The paper prints no such pattern; this composition is this build's stand-in for the family it names. */
void pretok_split3(const Text &t, std::vector<size_t> &starts) {
    const size_t n = t.cp.size();
    std::vector<std::pair<size_t, size_t>> a_spans, b_spans;
    for (size_t p = 0; p < n;) {                              /* A */
        size_t e = p;
        if (g_cls[t.cp[p]] == K_N) { while (e < n && e < p + 3 && g_cls[t.cp[e]] == K_N) e++; }
        else { while (e < n && g_cls[t.cp[e]] != K_N) e++; }
        a_spans.push_back({p, e});
        p = e;
    }
    for (auto sp : a_spans) {                                 /* B, inside every span of A */
        for (size_t p = sp.first; p < sp.second;) {
            const bool in = g_cls[t.cp[p]] == K_LB;
            size_t e = p;
            while (e < sp.second && (g_cls[t.cp[e]] == K_LB) == in) e++;
            b_spans.push_back({p, e});
            p = e;
        }
    }
    starts.clear();
    for (auto sp : b_spans) {                                 /* C: pattern 0 on the span alone */
        Text sub;
        sub.cp.assign(t.cp.begin() + sp.first, t.cp.begin() + sp.second);
        std::vector<size_t> st;
        pretok_plain(sub, 0, st);
        for (size_t x : st) starts.push_back(sp.first + x);
    }
}

void pretok_cp(const Text &t, int pattern, std::vector<size_t> &starts) {
    if (pattern == 3) pretok_split3(t, starts); else pretok_plain(t, pattern, starts);
}

/* ------------------------------------------------------------------------------- BPE */
struct Merge { int32_t left, right, result; };
struct Vocab {
    std::vector<Merge> merges;
    int32_t byte_map[256];
    std::unordered_map<uint64_t, int32_t> rank;    /* (left,right) -> rank (= index) */
    std::vector<std::string> token_bytes;          /* indexed by id (sparse ids allowed) */
    int32_t max_id = 0;
    /* Paper Sec. 4.2 (families configured with ignore_merges): the encoder emits a single id whenever the
     * whole piece is a vocabulary entry, whatever the merge loop would have made of its bytes.  Where two
     * entries spell the same bytes the one defined first (a base byte, else the lowest rank) is taken. */
    bool ignore_merges = false;
    std::unordered_map<std::string, int32_t> by_bytes;
};
inline uint64_t pair_key(int32_t a, int32_t b) { return ((uint64_t)(uint32_t)a << 32) | (uint32_t)b; }

/* Definition (paper Sec. 4.2 gives only schedules that must equal it): while some adjacent pair
 * is in the merge table, replace the lowest-ranked such pair, leftmost on ties, by its result. */
void bpe_naive(const Vocab &v, const uint8_t *b, size_t n, std::vector<int32_t> &t) {
    t.resize(n);
    for (size_t i = 0; i < n; i++) t[i] = v.byte_map[b[i]];
    for (;;) {
        int32_t best = INT32_MAX; size_t at = 0;
        for (size_t i = 0; i + 1 < t.size(); i++) {
            auto it = v.rank.find(pair_key(t[i], t[i + 1]));
            if (it != v.rank.end() && it->second < best) { best = it->second; at = i; }
        }
        if (best == INT32_MAX) return;
        t[at] = v.merges[best].result;
        t.erase(t.begin() + at + 1);
    }
}

/* Same definition with a linked list and a heap of (rank, position), for very long pieces. */
void bpe_heap(const Vocab &v, const uint8_t *b, size_t n, std::vector<int32_t> &out) {
    std::vector<int32_t> tok(n); std::vector<int64_t> prev(n), next(n); std::vector<char> alive(n, 1);
    for (size_t i = 0; i < n; i++) { tok[i] = v.byte_map[b[i]]; prev[i] = (int64_t)i - 1; next[i] = i + 1 < n ? (int64_t)i + 1 : -1; }
    struct E { int32_t rank; int64_t pos; int32_t l, r; };
    auto cmp = [](const E &a, const E &c) { return a.rank != c.rank ? a.rank > c.rank : a.pos > c.pos; };
    std::priority_queue<E, std::vector<E>, decltype(cmp)> pq(cmp);
    auto push = [&](int64_t i) {
        if (i < 0 || next[i] < 0) return;
        auto it = v.rank.find(pair_key(tok[i], tok[next[i]]));
        if (it != v.rank.end()) pq.push(E{it->second, i, tok[i], tok[next[i]]});
    };
    for (size_t i = 0; i < n; i++) push((int64_t)i);
    while (!pq.empty()) {
        E e = pq.top(); pq.pop();
        int64_t i = e.pos;
        if (!alive[i] || next[i] < 0 || tok[i] != e.l || tok[next[i]] != e.r) continue;   /* stale */
        int64_t j = next[i];
        tok[i] = v.merges[e.rank].result; alive[j] = 0;
        next[i] = next[j]; if (next[j] >= 0) prev[next[j]] = i;
        push(prev[i]); push(i);
    }
    out.clear();
    for (int64_t i = n ? 0 : -1; i >= 0; i = next[i]) out.push_back(tok[i]);
}

void bpe_piece(const Vocab &v, const uint8_t *b, size_t n, std::vector<int32_t> &t) {
    if (v.ignore_merges) {
        auto it = v.by_bytes.find(std::string((const char *)b, n));
        if (it != v.by_bytes.end()) { t.assign(1, it->second); return; }
    }
    if (n <= 2048) bpe_naive(v, b, n, t); else bpe_heap(v, b, n, t);
}

int64_t encode_impl(const Vocab &v, int pattern, const uint8_t *text, size_t len, int nthreads,
                    std::vector<int32_t> &ids, std::vector<int64_t> &piece_off) {
    Text t;
    if (!decode_utf8(text, len, t)) return -1;
    std::vector<size_t> starts;
    pretok_cp(t, pattern, starts);
    size_t P = starts.size();
    piece_off.resize(P + 1);
    for (size_t i = 0; i < P; i++) piece_off[i] = t.off[starts[i]];
    piece_off[P] = (int64_t)len;
    if (nthreads <= 1) {
        std::vector<int32_t> tmp;
        ids.clear();
        for (size_t i = 0; i < P; i++) {
            bpe_piece(v, text + piece_off[i], (size_t)(piece_off[i + 1] - piece_off[i]), tmp);
            ids.insert(ids.end(), tmp.begin(), tmp.end());
        }
    } else {
        /* pieces sharded across threads by equal byte ranges, results concatenated in order */
        std::vector<std::vector<int32_t>> part(nthreads);
        std::vector<std::thread> th;
        for (int k = 0; k < nthreads; k++) {
            th.emplace_back([&, k]() {
                size_t lo = P * k / nthreads, hi = P * (k + 1) / nthreads;
                std::vector<int32_t> tmp;
                for (size_t i = lo; i < hi; i++) {
                    bpe_piece(v, text + piece_off[i], (size_t)(piece_off[i + 1] - piece_off[i]), tmp);
                    part[k].insert(part[k].end(), tmp.begin(), tmp.end());
                }
            });
        }
        for (auto &x : th) x.join();
        ids.clear();
        for (auto &pp : part) ids.insert(ids.end(), pp.begin(), pp.end());
    }
    return (int64_t)ids.size();
}

}  // namespace

extern "C" {

void orc_set_class_table(const uint8_t *table) { g_cls = table; }

/* Returns the number of code points, or -1 for invalid UTF-8. */
int64_t orc_utf8_check(const uint8_t *text, size_t len) {
    Text t;
    return decode_utf8(text, len, t) ? (int64_t)t.cp.size() : -1;
}

/* Piece start BYTE offsets.  Returns the piece count (may exceed cap; only cap are written),
 * or -1 for invalid UTF-8. */
int64_t orc_pretok(int pattern, const uint8_t *text, size_t len, int64_t *starts_out, size_t cap) {
    Text t;
    if (!decode_utf8(text, len, t)) return -1;
    std::vector<size_t> st;
    pretok_cp(t, pattern, st);
    for (size_t i = 0; i < st.size() && i < cap; i++) starts_out[i] = t.off[st[i]];
    return (int64_t)st.size();
}

/* Piece starts of a batch: every document [doc_off[d], doc_off[d+1]) is matched exactly as if it were alone
 * (orc_pretok on its bytes); the starts are written as offsets into the concatenation, in document order.
 * Documents are spread over threads in contiguous ranges.  Returns the total piece count (only cap are
 * written), or -(d+1) if document d is invalid UTF-8. */
int64_t orc_pretok_batch(int pattern, const uint8_t *text, const int64_t *doc_off, size_t n_docs, int nthreads,
                         int64_t *starts_out, size_t cap) {
    if (nthreads < 1) nthreads = 1;
    std::vector<std::vector<int64_t>> part((size_t)nthreads);
    std::vector<int64_t> bad((size_t)nthreads, 0);
    std::vector<std::thread> th;
    const size_t per = (n_docs + (size_t)nthreads - 1) / (size_t)nthreads;
    for (int k = 0; k < nthreads; k++) {
        th.emplace_back([&, k]() {
            const size_t lo = std::min(n_docs, (size_t)k * per), hi = std::min(n_docs, lo + per);
            Text t; std::vector<size_t> st;
            for (size_t d = lo; d < hi; d++) {
                const size_t len = (size_t)(doc_off[d + 1] - doc_off[d]);
                if (!decode_utf8(text + doc_off[d], len, t)) { bad[k] = -(int64_t)(d + 1); return; }
                st.clear();
                pretok_cp(t, pattern, st);
                for (size_t i = 0; i < st.size(); i++) part[k].push_back(doc_off[d] + (int64_t)t.off[st[i]]);
            }
        });
    }
    for (auto &x : th) x.join();
    for (int k = 0; k < nthreads; k++) if (bad[k] < 0) return bad[k];
    size_t n = 0;
    for (auto &p : part) { for (int64_t v : p) { if (n < cap) starts_out[n] = v; n++; } }
    return (int64_t)n;
}

void *orc_vocab_new(const int32_t *merges /* n x 3: left,right,result */, size_t n, const int32_t *byte_map) {
    Vocab *v = new Vocab();
    std::memcpy(v->byte_map, byte_map, sizeof(v->byte_map));
    v->merges.resize(n);
    int32_t mx = 0;
    for (int i = 0; i < 256; i++) mx = std::max(mx, byte_map[i]);
    for (size_t i = 0; i < n; i++) {
        v->merges[i] = Merge{merges[3 * i], merges[3 * i + 1], merges[3 * i + 2]};
        mx = std::max(mx, merges[3 * i + 2]);
        v->rank.emplace(pair_key(merges[3 * i], merges[3 * i + 1]), (int32_t)i);   /* first occurrence wins */
    }
    v->max_id = mx;
    v->token_bytes.assign((size_t)mx + 1, std::string());
    std::vector<char> have((size_t)mx + 1, 0);
    for (int i = 0; i < 256; i++) if (byte_map[i] >= 0) { v->token_bytes[byte_map[i]] = std::string(1, (char)i); have[byte_map[i]] = 1; }
    for (size_t i = 0; i < n; i++) {
        const Merge &m = v->merges[i];
        if (m.left >= 0 && m.right >= 0 && m.left <= mx && m.right <= mx && m.result >= 0 && have[m.left] && have[m.right]) {
            v->token_bytes[m.result] = v->token_bytes[m.left] + v->token_bytes[m.right]; have[m.result] = 1;
        }
    }
    return v;
}
void orc_vocab_free(void *v) { delete (Vocab *)v; }

/* Switches the whole-piece rule on or off (off by default). */
void orc_vocab_set_ignore_merges(void *vp, int on) {
    Vocab *v = (Vocab *)vp;
    v->ignore_merges = on != 0;
    if (on && v->by_bytes.empty()) {
        for (int i = 0; i < 256; i++) if (v->byte_map[i] >= 0) v->by_bytes.emplace(std::string(1, (char)i), v->byte_map[i]);
        for (const Merge &m : v->merges)
            if (m.result >= 0 && m.result <= v->max_id && !v->token_bytes[m.result].empty())
                v->by_bytes.emplace(v->token_bytes[m.result], m.result);      /* emplace keeps the first */
    }
}

/* Byte string of a token id; returns its length (0 if unknown), writes up to cap bytes. */
size_t orc_token_bytes(const void *vp, int32_t id, uint8_t *out, size_t cap) {
    const Vocab *v = (const Vocab *)vp;
    if (id < 0 || id > v->max_id) return 0;
    const std::string &s = v->token_bytes[id];
    std::memcpy(out, s.data(), std::min(cap, s.size()));
    return s.size();
}

/* Byte lengths of n tokens (0 for an unknown id). */
void orc_token_lens(const void *vp, const int32_t *ids, size_t n, int64_t *out) {
    const Vocab *v = (const Vocab *)vp;
    for (size_t i = 0; i < n; i++) out[i] = (ids[i] < 0 || ids[i] > v->max_id) ? 0 : (int64_t)v->token_bytes[ids[i]].size();
}

/* BPE of one piece.  variant 0 = rescan (the definition), 1 = heap, 2 = by length. */
int64_t orc_bpe(const void *vp, const uint8_t *bytes, size_t n, int variant, int32_t *out, size_t cap) {
    std::vector<int32_t> t;
    if (variant == 0) bpe_naive(*(const Vocab *)vp, bytes, n, t);
    else if (variant == 1) bpe_heap(*(const Vocab *)vp, bytes, n, t);
    else bpe_piece(*(const Vocab *)vp, bytes, n, t);
    for (size_t i = 0; i < t.size() && i < cap; i++) out[i] = t[i];
    return (int64_t)t.size();
}

/* Whole path.  ids_out capacity ids_cap (len always suffices), piece_off_out capacity len+1 (may be
 * null).  Returns the token count or -1 for invalid UTF-8; *n_pieces receives the piece count. */
int64_t orc_encode(const void *vp, int pattern, const uint8_t *text, size_t len, int nthreads,
                   int32_t *ids_out, size_t ids_cap, int64_t *piece_off_out, int64_t *n_pieces) {
    std::vector<int32_t> ids; std::vector<int64_t> po;
    int64_t r = encode_impl(*(const Vocab *)vp, pattern, text, len, nthreads, ids, po);
    if (r < 0) { if (n_pieces) *n_pieces = 0; return -1; }
    for (size_t i = 0; i < ids.size() && i < ids_cap; i++) ids_out[i] = ids[i];
    if (piece_off_out) std::memcpy(piece_off_out, po.data(), po.size() * sizeof(int64_t));
    if (n_pieces) *n_pieces = (int64_t)po.size() - 1;
    return r;
}

/* Batch: every document is encoded exactly as if it were alone (paper Sec. 4.2: runs are cut at
 * document boundaries).  Documents are spread over threads.  ids_off_out has n_docs+1 entries.
 * Returns total tokens, or -(d+1) if document d is invalid UTF-8. */
int64_t orc_encode_batch(const void *vp, int pattern, const uint8_t *text, const int64_t *doc_off, size_t n_docs,
                         int nthreads, int32_t *ids_out, size_t ids_cap, int64_t *ids_off_out) {
    std::vector<std::vector<int32_t>> res(n_docs);
    std::vector<int64_t> rc(n_docs, 0);
    if (nthreads < 1) nthreads = 1;
    std::vector<std::thread> th;
    for (int k = 0; k < nthreads; k++) {
        th.emplace_back([&, k]() {
            std::vector<int64_t> po;
            for (size_t d = k; d < n_docs; d += nthreads)
                rc[d] = encode_impl(*(const Vocab *)vp, pattern, text + doc_off[d], (size_t)(doc_off[d + 1] - doc_off[d]), 1, res[d], po);
        });
    }
    for (auto &x : th) x.join();
    int64_t tot = 0;
    for (size_t d = 0; d < n_docs; d++) {
        if (rc[d] < 0) return -(int64_t)(d + 1);
        ids_off_out[d] = tot;
        for (size_t i = 0; i < res[d].size(); i++) if ((size_t)tot + i < ids_cap) ids_out[tot + i] = res[d][i];
        tot += (int64_t)res[d].size();
    }
    ids_off_out[n_docs] = tot;
    return tot;
}

/* ------------------------------------------------------------------------------ trainer
 * Standard BPE training on the distinct pieces of a corpus: repeatedly take the most frequent
 * adjacent pair (ties: smallest (left,right)), give it id 256+rank, and apply it everywhere.
 * Not part of the tokenization path; it only produces the merge lists the workloads use.
 * pairs_out: n_merges x 2.  Returns the number of merges produced. */
int64_t orc_train(int pattern, const uint8_t *corpus, size_t len, size_t n_merges, int32_t *pairs_out,
                  int64_t *n_distinct_out) {
    Text t;
    if (!decode_utf8(corpus, len, t)) return -1;
    std::vector<size_t> st;
    pretok_cp(t, pattern, st);
    std::unordered_map<std::string, int64_t> cnt;
    cnt.reserve(st.size() / 8 + 16);
    for (size_t i = 0; i < st.size(); i++) {
        int64_t a = t.off[st[i]], b = i + 1 < st.size() ? t.off[st[i + 1]] : (int64_t)len;
        cnt[std::string((const char *)corpus + a, (size_t)(b - a))]++;
    }
    t.cp.clear(); t.cp.shrink_to_fit(); t.off.clear(); t.off.shrink_to_fit();
    struct Word { std::vector<int32_t> tok; int64_t c; };
    std::vector<Word> words; words.reserve(cnt.size());
    {
        std::vector<std::pair<std::string, int64_t>> sorted(cnt.begin(), cnt.end());
        std::sort(sorted.begin(), sorted.end());      /* deterministic word order */
        cnt.clear();
        for (auto &kv : sorted) {
            if (kv.first.size() < 2) continue;
            Word w; w.c = kv.second; w.tok.resize(kv.first.size());
            for (size_t i = 0; i < kv.first.size(); i++) w.tok[i] = (uint8_t)kv.first[i];
            words.push_back(std::move(w));
        }
    }
    if (n_distinct_out) *n_distinct_out = (int64_t)words.size();
    std::unordered_map<uint64_t, int64_t> pc;
    std::unordered_map<uint64_t, std::vector<int32_t>> where;
    for (size_t wi = 0; wi < words.size(); wi++) {
        const Word &w = words[wi];
        for (size_t i = 0; i + 1 < w.tok.size(); i++) {
            uint64_t key = pair_key(w.tok[i], w.tok[i + 1]);
            pc[key] += w.c;
            auto &vec = where[key];
            if (vec.empty() || vec.back() != (int32_t)wi) vec.push_back((int32_t)wi);
        }
    }
    struct H { int64_t c; uint64_t key; };
    auto cmp = [](const H &a, const H &b) { return a.c != b.c ? a.c < b.c : a.key > b.key; };
    std::priority_queue<H, std::vector<H>, decltype(cmp)> pq(cmp);
    for (auto &kv : pc) pq.push(H{kv.second, kv.first});
    size_t done = 0;
    while (done < n_merges && !pq.empty()) {
        H top = pq.top(); pq.pop();
        auto it = pc.find(top.key);
        int64_t cur = it == pc.end() ? 0 : it->second;
        if (cur != top.c) { if (cur > 0) pq.push(H{cur, top.key}); continue; }
        if (cur <= 0) continue;
        int32_t L = (int32_t)(top.key >> 32), R = (int32_t)(top.key & 0xFFFFFFFFu), id = (int32_t)(256 + done);
        pairs_out[2 * done] = L; pairs_out[2 * done + 1] = R; done++;
        std::vector<int32_t> ws; ws.swap(where[top.key]);
        std::unordered_map<uint64_t, int64_t> delta;
        for (int32_t wi : ws) {
            Word &w = words[wi];
            std::vector<int32_t> &tk = w.tok;
            bool any = false;
            for (size_t i = 0; i + 1 < tk.size(); i++) if (tk[i] == L && tk[i + 1] == R) { any = true; break; }
            if (!any) continue;
            for (size_t i = 0; i + 1 < tk.size(); i++) delta[pair_key(tk[i], tk[i + 1])] -= w.c;
            std::vector<int32_t> nt; nt.reserve(tk.size());
            for (size_t i = 0; i < tk.size();) {
                if (i + 1 < tk.size() && tk[i] == L && tk[i + 1] == R) { nt.push_back(id); i += 2; }
                else nt.push_back(tk[i++]);
            }
            tk.swap(nt);
            for (size_t i = 0; i + 1 < tk.size(); i++) {
                uint64_t key = pair_key(tk[i], tk[i + 1]);
                delta[key] += w.c;
                if (tk[i] == id || tk[i + 1] == id) {
                    auto &vec = where[key];
                    if (vec.empty() || vec.back() != wi) vec.push_back(wi);
                }
            }
        }
        for (auto &kv : delta) {
            if (kv.second == 0) continue;
            int64_t &c = pc[kv.first];
            c += kv.second;
            if (c > 0) pq.push(H{c, kv.first});
        }
        pc.erase(top.key);
    }
    return (int64_t)done;
}

}  // extern "C"

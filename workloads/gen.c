/*
 * Seeded synthetic text generator for the tokenizer workloads.
 *
 * This file holds NO tokenizer arithmetic: it only draws pseudo-random text
 * (prose, Python-like code, JSON / log tool output, agent-transcript blocks,
 * non-ASCII words, adversarial long runs).  Both the CPU oracle tests and the
 * CUDA path read the bytes it writes; neither shares anything else.
 *
 * PRNG: splitmix64 seeding + xoshiro256**, implemented here so the byte
 * stream is a function of (kind, seed, n_chars) only.
 *
 * Kinds
 *   0  MIX          60 % prose / 30 % code / 10 % JSON, ASCII only, LF
 *   1  MIX_UNI      MIX + ~5 % non-ASCII code points + CRLF on 10 % of lines
 *   2  TRANSCRIPT   user/assistant/tool blocks, lognormal(median 1400, s=1.3)
 *                   block lengths, 40 % code / 30 % JSON+log / 30 % prose
 *   3  TRANSCRIPT_ADV  TRANSCRIPT + ~10 % CJK text + adversarial inserts
 *                   (64 KB space/tab runs, 20,000-digit strings, 50 KB runs
 *                   of one punctuation character)
 *
 * "chars" are Unicode code points; output is valid UTF-8 with exactly
 * n_chars code points.
 */
#include <stdint.h>
#include <stddef.h>
#include <stdlib.h>
#include <string.h>
#include <math.h>
#include <stdio.h>

/* ------------------------------------------------------------------ PRNG */
typedef struct { uint64_t s[4]; } rng_t;
static uint64_t splitmix64(uint64_t *x) {
    uint64_t z = (*x += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static void rng_seed(rng_t *r, uint64_t seed) {
    for (int i = 0; i < 4; i++) r->s[i] = splitmix64(&seed);
}
static inline uint64_t rotl(uint64_t x, int k) { return (x << k) | (x >> (64 - k)); }
static uint64_t rng_next(rng_t *r) {
    uint64_t *s = r->s;
    uint64_t result = rotl(s[1] * 5, 7) * 9, t = s[1] << 17;
    s[2] ^= s[0]; s[3] ^= s[1]; s[1] ^= s[2]; s[0] ^= s[3]; s[2] ^= t; s[3] = rotl(s[3], 45);
    return result;
}
static double rng_u01(rng_t *r) { return (double)(rng_next(r) >> 11) * (1.0 / 9007199254740992.0); }
static uint32_t rng_below(rng_t *r, uint32_t n) { return (uint32_t)(((rng_next(r) >> 32) * (uint64_t)n) >> 32); }
static int rng_chance(rng_t *r, double p) { return rng_u01(r) < p; }
static double rng_normal(rng_t *r) {
    double u1 = rng_u01(r), u2 = rng_u01(r);
    if (u1 < 1e-300) u1 = 1e-300;
    return sqrt(-2.0 * log(u1)) * cos(6.283185307179586 * u2);
}
static double rng_lognormal(rng_t *r, double median, double sigma) { return median * exp(sigma * rng_normal(r)); }

/* --------------------------------------------------------------- lexicon */
#define LEX_N 5000
#define LEX_MAXLEN 20
static char lex[LEX_N][LEX_MAXLEN];
static uint8_t lex_len[LEX_N];
static double zipf_cdf[LEX_N];
static int lex_ready = 0;

static const char *ONSET[] = {"b","c","d","f","g","h","j","k","l","m","n","p","r","s","t","v","w","z",
                              "br","ch","cl","dr","fl","gr","pl","pr","sh","st","th","tr","qu","sk"};
static const char *VOWEL[] = {"a","e","i","o","u","a","e","i","o","ai","ea","ou","io","ee"};
static const char *CODA[]  = {"","","","","n","r","s","t","l","m","x","ng","nd","st","ck"};

static void lex_init(void) {
    if (lex_ready) return;
    rng_t r; rng_seed(&r, 0x1E81C0DEull);
    int n = 0;
    while (n < LEX_N) {
        char w[64]; int len = 0;
        int nsyl = 2 + (int)rng_below(&r, 3);
        if (n < 60) nsyl = 1;                /* a few very short, very frequent words */
        for (int k = 0; k < nsyl; k++) {
            const char *o = ONSET[rng_below(&r, sizeof(ONSET) / sizeof(*ONSET))];
            const char *v = VOWEL[rng_below(&r, sizeof(VOWEL) / sizeof(*VOWEL))];
            const char *c = CODA[rng_below(&r, sizeof(CODA) / sizeof(*CODA))];
            if (k == 0 && rng_chance(&r, 0.2)) o = "";
            len += sprintf(w + len, "%s%s%s", o, v, c);
        }
        if (len >= LEX_MAXLEN || len < 1) continue;
        int dup = 0;
        for (int i = 0; i < n && !dup; i++) dup = (lex_len[i] == len && memcmp(lex[i], w, len) == 0);
        if (dup) continue;
        memcpy(lex[n], w, len); lex[n][len] = 0; lex_len[n] = (uint8_t)len; n++;
    }
    double tot = 0;
    for (int i = 0; i < LEX_N; i++) { tot += pow(i + 1.0, -1.1); zipf_cdf[i] = tot; }
    for (int i = 0; i < LEX_N; i++) zipf_cdf[i] /= tot;
    lex_ready = 1;
}
static int zipf_word(rng_t *r) {
    double u = rng_u01(r);
    int lo = 0, hi = LEX_N - 1;
    while (lo < hi) { int mid = (lo + hi) >> 1; if (zipf_cdf[mid] < u) lo = mid + 1; else hi = mid; }
    return lo;
}

/* ---------------------------------------------------------------- buffer */
typedef struct {
    uint8_t *p; size_t len, cap; size_t chars;
    rng_t rng;
    double uni_rate;    /* probability that a prose word is replaced by a non-ASCII item */
    double crlf_rate;   /* probability that a line ends in CRLF */
    double cjk_rate;    /* probability that a prose paragraph is CJK */
    int line_crlf;
    int adv_next;
} ctx_t;

static void put_bytes(ctx_t *c, const void *s, size_t n, size_t nchars) {
    if (c->len + n + 8 > c->cap) {
        size_t nc = c->cap * 2 + n + 64;
        c->p = (uint8_t *)realloc(c->p, nc); c->cap = nc;
    }
    memcpy(c->p + c->len, s, n); c->len += n; c->chars += nchars;
}
static void put_s(ctx_t *c, const char *s) { size_t n = strlen(s); put_bytes(c, s, n, n); }
static void put_c(ctx_t *c, char ch) { put_bytes(c, &ch, 1, 1); }
static void put_cp(ctx_t *c, uint32_t cp) {
    uint8_t b[4]; size_t n;
    if (cp < 0x80) { b[0] = (uint8_t)cp; n = 1; }
    else if (cp < 0x800) { b[0] = 0xC0 | (cp >> 6); b[1] = 0x80 | (cp & 63); n = 2; }
    else if (cp < 0x10000) { b[0] = 0xE0 | (cp >> 12); b[1] = 0x80 | ((cp >> 6) & 63); b[2] = 0x80 | (cp & 63); n = 3; }
    else { b[0] = 0xF0 | (cp >> 18); b[1] = 0x80 | ((cp >> 12) & 63); b[2] = 0x80 | ((cp >> 6) & 63); b[3] = 0x80 | (cp & 63); n = 4; }
    put_bytes(c, b, n, 1);
}
static void put_nl(ctx_t *c) {
    if (c->line_crlf) put_s(c, "\r\n"); else put_c(c, '\n');
    c->line_crlf = rng_chance(&c->rng, c->crlf_rate);
}
static void put_word(ctx_t *c, int w, int cap_mode) {   /* 0 lower, 1 Capitalised, 2 UPPER */
    char t[LEX_MAXLEN]; int n = lex_len[w];
    memcpy(t, lex[w], n);
    if (cap_mode >= 1) t[0] = (char)(t[0] - 32);
    if (cap_mode == 2) for (int i = 1; i < n; i++) t[i] = (char)(t[i] - 32);
    put_bytes(c, t, n, n);
}
static void put_int(ctx_t *c, uint64_t v) { char t[32]; int n = sprintf(t, "%llu", (unsigned long long)v); put_bytes(c, t, n, n); }
static uint64_t log_uniform_int(rng_t *r, double hi) {   /* integers roughly uniform in log space over [0, hi] */
    double x = exp(rng_u01(r) * log(hi + 1.0)) - 1.0;
    return (uint64_t)x;
}

/* ------------------------------------------------------- non-ASCII items */
static const uint32_t ACCENT[] = {0xE9,0xE8,0xEA,0xE1,0xE0,0xE4,0xF6,0xFC,0xF1,0xE7,0xED,0xF3,0xFA,0xDF,0xC9,0xD6,0x159,0x142,0x11B};
static const uint32_t CJK_PUNCT[] = {0x3002, 0xFF0C, 0x3001, 0xFF01, 0xFF1F};
static uint32_t cjk_char(rng_t *r) {
    /* Zipf-like over the 20,992 unified ideographs so that frequent characters repeat */
    double u = rng_u01(r);
    uint32_t k = (uint32_t)(20992.0 * u * u * u);
    if (k >= 20992) k = 20991;
    return 0x4E00 + (k * 7919u) % 20992u;
}
static void put_accented_word(ctx_t *c) {
    int w = zipf_word(&c->rng); int n = lex_len[w];
    int cap = rng_chance(&c->rng, 0.15);
    int hit = 0;
    for (int i = 0; i < n; i++) {
        char ch = lex[w][i];
        int vowel = (ch == 'a' || ch == 'e' || ch == 'i' || ch == 'o' || ch == 'u');
        if ((vowel && rng_chance(&c->rng, 0.5)) || (i == n - 1 && !hit)) {
            uint32_t a = ACCENT[rng_below(&c->rng, sizeof(ACCENT) / sizeof(*ACCENT))];
            if (i == 0 && cap && a >= 0xE0 && a <= 0xFE && a != 0xF7) a -= 0x20;
            put_cp(c, a); hit = 1;
        } else put_c(c, (i == 0 && cap) ? (char)(ch - 32) : ch);
    }
}
static void put_cyrillic_word(ctx_t *c) {
    int n = 2 + (int)rng_below(&c->rng, 8);
    int cap = rng_chance(&c->rng, 0.2);
    for (int i = 0; i < n; i++) {
        uint32_t k = rng_below(&c->rng, 32);
        put_cp(c, (i == 0 && cap) ? 0x410 + k : 0x430 + k);
    }
}
static void put_cjk_run(ctx_t *c, int n) { for (int i = 0; i < n; i++) put_cp(c, cjk_char(&c->rng)); }
static void put_emoji(ctx_t *c) {
    uint32_t k = rng_below(&c->rng, 3);
    if (k == 0) put_cp(c, 0x1F600 + rng_below(&c->rng, 80));
    else if (k == 1) put_cp(c, 0x1F300 + rng_below(&c->rng, 256));
    else put_cp(c, 0x2600 + rng_below(&c->rng, 64));
}
static void put_unicode_item(ctx_t *c) {
    uint32_t k = rng_below(&c->rng, 100);
    if (k < 40) put_accented_word(c);
    else if (k < 65) put_cyrillic_word(c);
    else if (k < 90) put_cjk_run(c, 1 + (int)rng_below(&c->rng, 8));
    else put_emoji(c);
}

/* ------------------------------------------------------------------ prose */
static const char *CONTR[] = {"n't", "'s", "'re", "'ll", "'ve", "'d", "'m", "'S", "'T"};
static void emit_sentence(ctx_t *c) {
    int nw = 4 + (int)rng_below(&c->rng, 18);
    for (int i = 0; i < nw; i++) {
        if (i) put_c(c, ' ');
        if (rng_chance(&c->rng, c->uni_rate)) { put_unicode_item(c); continue; }
        if (rng_chance(&c->rng, 0.03)) { put_int(c, log_uniform_int(&c->rng, 1e7)); continue; }
        int w = zipf_word(&c->rng);
        int cap = (i == 0) ? 1 : (rng_chance(&c->rng, 0.04) ? 1 : (rng_chance(&c->rng, 0.01) ? 2 : 0));
        int quoted = rng_chance(&c->rng, 0.02);
        if (quoted) put_c(c, rng_chance(&c->rng, 0.5) ? '"' : '\'');
        put_word(c, w, cap);
        if (rng_chance(&c->rng, 0.03)) put_s(c, CONTR[rng_below(&c->rng, sizeof(CONTR) / sizeof(*CONTR))]);
        if (quoted) put_c(c, rng_chance(&c->rng, 0.5) ? '"' : '\'');
        if (i + 1 < nw) {
            uint32_t k = rng_below(&c->rng, 100);
            if (k < 8) put_c(c, ','); else if (k < 10) put_c(c, ';'); else if (k < 11) put_c(c, ':');
            else if (k < 12) put_s(c, " -"); else if (k < 13) put_s(c, " (");
        }
    }
    uint32_t k = rng_below(&c->rng, 100);
    put_s(c, k < 80 ? "." : k < 88 ? "?" : k < 94 ? "!" : k < 97 ? "..." : ")." );
}
static void emit_cjk_sentence(ctx_t *c) {
    int nseg = 1 + (int)rng_below(&c->rng, 7);
    for (int s = 0; s < nseg; s++) {
        put_cjk_run(c, 2 + (int)rng_below(&c->rng, 14));
        uint32_t k = rng_below(&c->rng, 100);
        if (k < 12) { put_word(c, zipf_word(&c->rng), 2); }                     /* ASCII acronym glued to CJK */
        else if (k < 20) { put_word(c, zipf_word(&c->rng), 1); }
        else if (k < 26) { put_int(c, log_uniform_int(&c->rng, 1e5)); }
        else if (k < 32) { put_c(c, ' '); put_word(c, zipf_word(&c->rng), 0); put_c(c, ' '); }
        if (s + 1 < nseg) put_cp(c, CJK_PUNCT[1 + rng_below(&c->rng, 2)]);
    }
    put_cp(c, CJK_PUNCT[rng_chance(&c->rng, 0.8) ? 0 : 3 + rng_below(&c->rng, 2)]);
}
static void emit_prose(ctx_t *c, size_t target_chars) {
    size_t end = c->chars + target_chars;
    while (c->chars < end) {
        int cjk = rng_chance(&c->rng, c->cjk_rate);
        int ns = 1 + (int)rng_below(&c->rng, 6);
        for (int i = 0; i < ns; i++) {
            if (cjk) emit_cjk_sentence(c);
            else { if (i) put_c(c, ' '); emit_sentence(c); }
        }
        put_nl(c);
        if (rng_chance(&c->rng, 0.6)) put_nl(c);
    }
}

/* ------------------------------------------------------------------- code */
static void put_ident(ctx_t *c, int style) {   /* 0 snake, 1 camel, 2 Pascal, 3 CONST */
    int nw = 1 + (int)rng_below(&c->rng, 3);
    for (int i = 0; i < nw; i++) {
        int w = zipf_word(&c->rng);
        if (style == 0) { if (i) put_c(c, '_'); put_word(c, w, 0); }
        else if (style == 1) put_word(c, w, i ? 1 : 0);
        else if (style == 2) put_word(c, w, 1);
        else { if (i) put_c(c, '_'); put_word(c, w, 2); }
    }
}
static int ident_style(ctx_t *c) {
    uint32_t k = rng_below(&c->rng, 100);
    return k < 55 ? 0 : k < 80 ? 1 : k < 93 ? 2 : 3;
}
static void put_string_lit(ctx_t *c) {
    char q = rng_chance(&c->rng, 0.6) ? '"' : '\'';
    put_c(c, q);
    int nw = 1 + (int)rng_below(&c->rng, 4);
    for (int i = 0; i < nw; i++) {
        if (i) put_c(c, rng_chance(&c->rng, 0.8) ? ' ' : '/');
        if (rng_chance(&c->rng, c->uni_rate)) put_unicode_item(c);
        else put_word(c, zipf_word(&c->rng), rng_chance(&c->rng, 0.1));
    }
    put_c(c, q);
}
static void put_expr(ctx_t *c, int depth) {
    uint32_t k = rng_below(&c->rng, 100);
    if (k < 30) put_ident(c, ident_style(c));
    else if (k < 45) put_int(c, log_uniform_int(&c->rng, 1e7));
    else if (k < 50) { put_int(c, rng_below(&c->rng, 1000)); put_c(c, '.'); put_int(c, rng_below(&c->rng, 10000)); }
    else if (k < 60) put_string_lit(c);
    else if (k < 75 && depth < 3) {
        put_ident(c, ident_style(c)); put_c(c, '(');
        int na = (int)rng_below(&c->rng, 4);
        for (int i = 0; i < na; i++) { if (i) put_s(c, ", "); put_expr(c, depth + 1); }
        put_c(c, ')');
    } else if (k < 88 && depth < 3) {
        static const char *OPS[] = {" + ", " - ", " * ", " / ", " == ", " != ", " <= ", " >= ", " and ", " or ", " % ", " // ", " << ", "**"};
        put_expr(c, depth + 1); put_s(c, OPS[rng_below(&c->rng, sizeof(OPS) / sizeof(*OPS))]); put_expr(c, depth + 1);
    } else if (k < 94) {
        put_ident(c, 0); put_c(c, '.'); put_ident(c, ident_style(c));
    } else if (depth < 3) {
        put_ident(c, 0); put_c(c, '['); put_expr(c, depth + 1); put_c(c, ']');
    } else put_ident(c, 0);
}
static void put_indent(ctx_t *c, int depth) { for (int i = 0; i < depth * 4; i++) put_c(c, ' '); }
static void emit_code(ctx_t *c, size_t target_chars) {
    size_t end = c->chars + target_chars;
    int depth = 0;
    while (c->chars < end) {
        uint32_t k = rng_below(&c->rng, 100);
        if (k < 8) { put_nl(c); continue; }
        if (k < 16 && depth > 0) depth -= 1 + (depth > 1 && rng_chance(&c->rng, 0.3));
        put_indent(c, depth);
        if (k < 26) {
            put_s(c, rng_chance(&c->rng, 0.8) ? "def " : "class "); put_ident(c, rng_chance(&c->rng, 0.7) ? 0 : 2); put_c(c, '(');
            int na = (int)rng_below(&c->rng, 4);
            for (int i = 0; i < na; i++) { if (i) put_s(c, ", "); put_ident(c, 0); if (rng_chance(&c->rng, 0.3)) { put_s(c, "="); put_expr(c, 2); } }
            put_s(c, "):"); if (depth < 6) depth++;
        } else if (k < 36) { put_s(c, rng_chance(&c->rng, 0.7) ? "if " : "while "); put_expr(c, 1); put_c(c, ':'); if (depth < 6) depth++; }
        else if (k < 42) { put_s(c, "for "); put_ident(c, 0); put_s(c, " in "); put_expr(c, 1); put_c(c, ':'); if (depth < 6) depth++; }
        else if (k < 50) { put_s(c, "return "); put_expr(c, 0); }
        else if (k < 58) { put_s(c, "# "); emit_sentence(c); }
        else if (k < 62) { put_s(c, rng_chance(&c->rng, 0.5) ? "import " : "from "); put_ident(c, 0); if (rng_chance(&c->rng, 0.5)) { put_s(c, " import "); put_ident(c, ident_style(c)); } }
        else if (k < 66) { put_s(c, "print(f\"{"); put_ident(c, 0); put_s(c, "}: {"); put_expr(c, 2); put_s(c, "}\")"); }
        else if (k < 70) { put_ident(c, 0); put_s(c, " = {"); int n = 1 + (int)rng_below(&c->rng, 3); for (int i = 0; i < n; i++) { if (i) put_s(c, ", "); put_string_lit(c); put_s(c, ": "); put_expr(c, 2); } put_c(c, '}'); }
        else if (k < 73) { put_s(c, "else:"); if (depth < 6) depth++; }
        else if (k < 75) { put_s(c, "\tassert "); put_expr(c, 1); put_s(c, "  "); }   /* stray tab + trailing blanks */
        else { put_ident(c, 0); static const char *AS[] = {" = ", " += ", " -= ", " |= ", ": int = "}; put_s(c, AS[rng_below(&c->rng, 5)]); put_expr(c, 0); }
        put_nl(c);
    }
}

/* ------------------------------------------------------------ JSON / logs */
static void put_json_value(ctx_t *c, int depth, int indent);
static void put_json_key(ctx_t *c) { put_c(c, '"'); put_ident(c, rng_chance(&c->rng, 0.6) ? 0 : 1); put_s(c, "\": "); }
static void put_path(ctx_t *c) {
    int n = 1 + (int)rng_below(&c->rng, 4);
    for (int i = 0; i < n; i++) { put_c(c, '/'); put_ident(c, 0); }
    static const char *EXT[] = {".py", ".json", ".txt", ".rs", ".log", ""};
    put_s(c, EXT[rng_below(&c->rng, 6)]);
}
static void put_timestamp(ctx_t *c) {
    char t[40];
    int n = sprintf(t, "20%02u-%02u-%02uT%02u:%02u:%02u.%03uZ", 20 + rng_below(&c->rng, 7), 1 + rng_below(&c->rng, 12), 1 + rng_below(&c->rng, 28),
                    rng_below(&c->rng, 24), rng_below(&c->rng, 60), rng_below(&c->rng, 60), rng_below(&c->rng, 1000));
    put_bytes(c, t, n, n);
}
static void put_hex(ctx_t *c, int n) { for (int i = 0; i < n; i++) put_c(c, "0123456789abcdef"[rng_below(&c->rng, 16)]); }
static void put_json_value(ctx_t *c, int depth, int indent) {
    uint32_t k = rng_below(&c->rng, 100);
    if (k < 35) put_int(c, log_uniform_int(&c->rng, 1e7));
    else if (k < 45) put_s(c, rng_chance(&c->rng, 0.5) ? "true" : rng_chance(&c->rng, 0.5) ? "false" : "null");
    else if (k < 60) put_string_lit(c);
    else if (k < 66) { put_c(c, '"'); put_path(c); put_c(c, '"'); }
    else if (k < 71) { put_c(c, '"'); put_timestamp(c); put_c(c, '"'); }
    else if (k < 75) { put_c(c, '"'); put_hex(c, 8 + 8 * (int)rng_below(&c->rng, 4)); put_c(c, '"'); }
    else if (k < 78) { put_c(c, '-'); put_int(c, rng_below(&c->rng, 1000)); put_c(c, '.'); put_int(c, rng_below(&c->rng, 100000)); }
    else if (k < 90 && depth < 4) {
        int n = 1 + (int)rng_below(&c->rng, 5);
        int multi = indent >= 0;
        put_c(c, '{');
        for (int i = 0; i < n; i++) {
            if (i) put_c(c, ',');
            if (multi) { put_nl(c); for (int s = 0; s < (indent + 1) * 2; s++) put_c(c, ' '); } else if (i) put_c(c, ' ');
            put_json_key(c); put_json_value(c, depth + 1, multi ? indent + 1 : -1);
        }
        if (multi) { put_nl(c); for (int s = 0; s < indent * 2; s++) put_c(c, ' '); }
        put_c(c, '}');
    } else if (depth < 4) {
        int n = (int)rng_below(&c->rng, 7);
        put_c(c, '[');
        for (int i = 0; i < n; i++) { if (i) put_s(c, ", "); put_json_value(c, depth + 2, -1); }
        put_c(c, ']');
    } else put_int(c, rng_below(&c->rng, 100));
}
static void emit_json(ctx_t *c, size_t target_chars) {
    size_t end = c->chars + target_chars;
    while (c->chars < end) {
        int pretty = rng_chance(&c->rng, 0.6);
        int n = 2 + (int)rng_below(&c->rng, 8);
        put_c(c, '{');
        for (int i = 0; i < n; i++) {
            if (i) put_c(c, ',');
            if (pretty) { put_nl(c); put_s(c, "  "); } else if (i) put_c(c, ' ');
            put_json_key(c); put_json_value(c, 1, pretty ? 1 : -1);
        }
        if (pretty) put_nl(c);
        put_c(c, '}'); put_nl(c);
    }
}
static void emit_log(ctx_t *c, size_t target_chars) {
    size_t end = c->chars + target_chars;
    static const char *LV[] = {"INFO", "DEBUG", "WARN", "ERROR", "TRACE"};
    while (c->chars < end) {
        uint32_t k = rng_below(&c->rng, 100);
        if (k < 70) {
            put_timestamp(c); put_c(c, ' '); put_s(c, LV[rng_below(&c->rng, 5)]); put_s(c, " ["); put_ident(c, 0); put_s(c, "] ");
            emit_sentence(c);
            if (rng_chance(&c->rng, 0.4)) { put_c(c, ' '); put_ident(c, 0); put_c(c, '='); put_int(c, log_uniform_int(&c->rng, 1e7)); }
            if (rng_chance(&c->rng, 0.2)) { put_s(c, " path="); put_path(c); }
        } else if (k < 80) {
            put_s(c, "  File \""); put_path(c); put_s(c, "\", line "); put_int(c, 1 + rng_below(&c->rng, 3000)); put_s(c, ", in "); put_ident(c, 0);
        } else if (k < 88) {
            put_s(c, "$ "); put_ident(c, 0); put_s(c, " --"); put_ident(c, 0); put_c(c, ' '); put_path(c);
        } else if (k < 94) {
            int n = 3 + (int)rng_below(&c->rng, 40); char ch = "-=*#~"[rng_below(&c->rng, 5)];
            for (int i = 0; i < n; i++) put_c(c, ch);
        } else {
            put_int(c, rng_below(&c->rng, 5000)); put_s(c, " passed, "); put_int(c, rng_below(&c->rng, 50)); put_s(c, " failed in ");
            put_int(c, rng_below(&c->rng, 300)); put_c(c, '.'); put_int(c, rng_below(&c->rng, 100)); put_c(c, 's');
        }
        put_nl(c);
    }
}

/* ------------------------------------------------------------ adversarial */
static void emit_adversarial(ctx_t *c) {
    uint32_t k = (uint32_t)(c->adv_next++ % 3);   /* round-robin so every kind appears */
    if (k == 0) {                                   /* 64 KB of spaces and tabs */
        uint32_t mode = rng_below(&c->rng, 3);
        if (rng_chance(&c->rng, 0.5)) put_c(c, '\n');
        for (int i = 0; i < 65536; i++) put_c(c, mode == 0 ? ' ' : mode == 1 ? '\t' : (rng_chance(&c->rng, 0.5) ? ' ' : '\t'));
    } else if (k == 1) {                            /* 20,000-digit number */
        for (int i = 0; i < 20000; i++) put_c(c, (char)('0' + rng_below(&c->rng, 10)));
    } else {                                        /* 50 KB of one punctuation character */
        char ch = "/'=-*#.!"[rng_below(&c->rng, 8)];
        if (rng_chance(&c->rng, 0.3)) put_s(c, ";\n");
        for (int i = 0; i < 51200; i++) put_c(c, ch);
    }
    uint32_t t = rng_below(&c->rng, 4);
    if (t == 0) put_nl(c); else if (t == 1) put_c(c, ' '); else if (t == 2) put_ident(c, 1);
}

/* ------------------------------------------------- mark-dense, blank-free text */
/* Latin letters with a combining mark after every second or third one, no blanks: words are glued, a comma or a full
 * stop comes every 20-80 characters and a line feed every few hundred. */
static void emit_marks(ctx_t *c, size_t n_chars) {
    static const uint32_t MARK[] = {0x301, 0x300, 0x308, 0x323, 0x302, 0x303};
    size_t next_punct = 20 + rng_below(&c->rng, 60), next_nl = 200 + rng_below(&c->rng, 300), since_mark = 0;
    while (c->chars < n_chars) {
        int upper = rng_chance(&c->rng, 0.06);
        put_c(c, (char)((upper ? 'A' : 'a') + rng_below(&c->rng, 26)));
        if (++since_mark >= 2 + rng_below(&c->rng, 2)) { put_cp(c, MARK[rng_below(&c->rng, 6)]); since_mark = 0; }
        if (rng_chance(&c->rng, 0.004)) { put_c(c, '\''); put_c(c, "stmd"[rng_below(&c->rng, 4)]); }
        if (c->chars >= next_punct) { put_c(c, rng_chance(&c->rng, 0.7) ? ',' : '.'); next_punct = c->chars + 20 + rng_below(&c->rng, 60); }
        if (c->chars >= next_nl) { put_c(c, '\n'); next_nl = c->chars + 200 + rng_below(&c->rng, 300); }
    }
}
/* Thai-like text: consonants (caseless letters, three bytes each) carrying vowel signs and tone marks (marks) above and
 * below, words glued into phrases of 5-40 characters that a single blank separates, now and then digits, a Latin
 * word or punctuation. */
static void emit_thai_like(ctx_t *c, size_t n_chars) {
    static const uint32_t SIGN[] = {0xE31, 0xE34, 0xE35, 0xE36, 0xE37, 0xE38, 0xE39, 0xE47, 0xE48, 0xE49, 0xE4A, 0xE4B, 0xE4C};
    lex_init();
    while (c->chars < n_chars) {
        size_t phrase = 5 + rng_below(&c->rng, 36);
        for (size_t k = 0; k < phrase; k++) {
            put_cp(c, 0xE01 + rng_below(&c->rng, 46));                       /* consonant */
            if (rng_chance(&c->rng, 0.45)) put_cp(c, SIGN[rng_below(&c->rng, 13)]);
            if (rng_chance(&c->rng, 0.12)) put_cp(c, 0xE30 + 2 * rng_below(&c->rng, 2));   /* a spacing vowel (letter) */
        }
        uint32_t k = rng_below(&c->rng, 100);
        if (k < 70) put_c(c, ' ');
        else if (k < 78) { put_c(c, ' '); put_int(c, log_uniform_int(&c->rng, 1e7)); put_c(c, ' '); }
        else if (k < 86) { put_c(c, ' '); put_word(c, zipf_word(&c->rng), rng_below(&c->rng, 3)); put_c(c, ' '); }
        else if (k < 94) put_s(c, rng_chance(&c->rng, 0.5) ? " (" : ") ");
        else put_nl(c);
    }
}

/* ------------------------------------------------------------- top level */
static void emit_mix(ctx_t *c, size_t n_chars) {
    while (c->chars < n_chars) {
        size_t chunk = 200 + rng_below(&c->rng, 1200);
        uint32_t k = rng_below(&c->rng, 100);
        if (k < 60) emit_prose(c, chunk); else if (k < 90) emit_code(c, chunk); else emit_json(c, chunk);
    }
}
static void emit_transcript(ctx_t *c, size_t n_chars, int adversarial) {
    static const char *ROLE[] = {"user", "assistant", "tool"};
    int turn = 0;
    while (c->chars < n_chars) {
        double len = rng_lognormal(&c->rng, 1400.0, 1.3);
        if (len < 40) len = 40; if (len > 400000) len = 400000;
        put_s(c, "<|"); put_s(c, ROLE[turn % 3]); put_s(c, "|>"); put_nl(c);
        uint32_t k = rng_below(&c->rng, 100);
        if (k < 40) {
            if (rng_chance(&c->rng, 0.5)) { put_s(c, "```python"); put_nl(c); emit_code(c, (size_t)len); put_s(c, "```"); put_nl(c); }
            else emit_code(c, (size_t)len);
        } else if (k < 55) emit_json(c, (size_t)len);
        else if (k < 70) emit_log(c, (size_t)len);
        else emit_prose(c, (size_t)len);
        if (adversarial && rng_chance(&c->rng, 0.012)) emit_adversarial(c);
        put_nl(c);
        turn++;
    }
}

static size_t truncate_to_chars(const uint8_t *p, size_t len, size_t n_chars) {
    size_t chars = 0, i = 0;
    while (i < len) {
        if ((p[i] & 0xC0) != 0x80) { if (chars == n_chars) break; chars++; }
        i++;
    }
    return i;
}

/* Generate exactly n_chars code points.  Returns the number of bytes written to `out`
 * (0 if cap is too small; 4*n_chars always suffices). */
size_t wl_generate(int kind, uint64_t seed, size_t n_chars, uint8_t *out, size_t cap) {
    lex_init();
    ctx_t c; memset(&c, 0, sizeof(c));
    c.cap = n_chars + n_chars / 4 + 4096; c.p = (uint8_t *)malloc(c.cap);
    rng_seed(&c.rng, seed ^ (0xA5A5A5A5ull * (uint64_t)(kind + 1)));
    if (kind == 1) { c.uni_rate = 0.17; c.crlf_rate = 0.10; }
    if (kind == 3) { c.uni_rate = 0.02; c.cjk_rate = 0.85; }
    if (kind == 0 || kind == 1) emit_mix(&c, n_chars);
    else if (kind == 4) emit_marks(&c, n_chars);
    else if (kind == 5) emit_thai_like(&c, n_chars);
    else emit_transcript(&c, n_chars, kind == 3);
    size_t nbytes = truncate_to_chars(c.p, c.len, n_chars);
    if (nbytes > cap) { free(c.p); return 0; }
    memcpy(out, c.p, nbytes);
    free(c.p);
    return nbytes;
}

/* Lognormal request lengths (in chars) for a batch, clipped to [lo, hi]. */
void wl_batch_lengths(uint64_t seed, size_t n, double median, double sigma, double lo, double hi, uint64_t *out) {
    rng_t r; rng_seed(&r, seed);
    for (size_t i = 0; i < n; i++) {
        double v = rng_lognormal(&r, median, sigma);
        if (v < lo) v = lo; if (v > hi) v = hi;
        out[i] = (uint64_t)v;
    }
}

/* Count code points (non-continuation bytes). */
size_t wl_count_chars(const uint8_t *p, size_t len) {
    size_t n = 0;
    for (size_t i = 0; i < len; i++) n += ((p[i] & 0xC0) != 0x80);
    return n;
}

/* Every string of 1..maxlen symbols over an alphabet of k symbols (each symbol a byte string of its own,
 * sym_off[k+1] offsets into sym_bytes), shortest first, each length in odometer order with the last
 * position fastest.  The strings are written back to back into `out`; doc_off receives the n + 1 byte
 * offsets.  Returns the number of strings n, or 0 if either buffer is too small.  With out == NULL only
 * the sizes are computed: *bytes_needed receives the total number of bytes. */
size_t wl_exhaustive(const uint8_t *sym_bytes, const uint32_t *sym_off, int k, int maxlen, uint8_t *out, size_t cap,
                     int64_t *doc_off, size_t doc_cap, size_t *bytes_needed) {
    size_t n = 0, bytes = 0;
    int idx[32];
    if (k < 1 || maxlen < 1 || maxlen > 32) return 0;
    for (int len = 1; len <= maxlen; len++) {
        for (int i = 0; i < len; i++) idx[i] = 0;
        for (;;) {
            if (out) {
                if (n + 1 >= doc_cap) return 0;
                doc_off[n] = (int64_t)bytes;
            }
            for (int i = 0; i < len; i++) {
                const uint32_t a = sym_off[idx[i]], b = sym_off[idx[i] + 1];
                if (out) { if (bytes + (b - a) > cap) return 0; memcpy(out + bytes, sym_bytes + a, b - a); }
                bytes += b - a;
            }
            n++;
            int i = len - 1;
            while (i >= 0 && ++idx[i] == k) { idx[i] = 0; i--; }
            if (i < 0) break;
        }
    }
    if (out) doc_off[n] = (int64_t)bytes;
    if (bytes_needed) *bytes_needed = bytes;
    return n;
}

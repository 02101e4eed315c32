/*
 * toktier.h -- C ABI of the B200 (sm_100a) exact full-request tokenizer.
 *
 * The library computes, entirely in CUDA kernels, what the paper's Sec. 4 ("Exact GPU
 * Tokenization") describes: GPT-family regex pre-tokenization re-expressed as per-character
 * class tags, maximal runs and a run-local piece-start predicate (Sec. 4.1), followed by
 * byte-level BPE applied to every piece independently (Sec. 4.2), with counts kept on the
 * device so that no call synchronises with the host (Sec. 4.3).  Output token IDs are identical
 * to sequential leftmost-first matching followed by lowest-rank-first merging.
 *
 * Conventions
 *   - "DEVICE" pointers are CUDA device addresses on the current device; "HOST" pointers are
 *     ordinary host addresses.  The library never frees or reallocates caller memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Every tt_encode* / tt_pretokenize call only enqueues work on `stream`; it never
 *     synchronises and never reads device memory on the host.  Data-dependent failures are
 *     reported through the DEVICE status word (see below), never by trapping.
 *   - Host return value: TT_OK or a TT_ERR_* code describing an argument / CUDA problem.
 *   - There is no CPU fallback: without a CUDA device the calls fail with TT_ERR_CUDA.
 */
#ifndef TOKTIER_H
#define TOKTIER_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* host return codes and device status values */
enum {
    TT_OK = 0,
    TT_ERR_ARG = 1,              /* null pointer, bad pattern id, buffer too small (host-detectable)   */
    TT_ERR_BAD_VOCAB = 2,        /* merge table rejected by tt_vocab_load                              */
    TT_ERR_CUDA = 3,             /* a CUDA runtime call failed (no device, out of memory, launch)      */
    TT_ERR_INVALID_UTF8 = 4,     /* device status: input is not strict UTF-8; zero tokens are returned */
    TT_ERR_CAPACITY = 5,         /* device status: ids_cap too small for the result; zero tokens       */
    TT_ERR_INTERNAL_TIMEOUT = 6, /* device status: a bounded device-side loop gave up                  */
    TT_ERR_TOO_LARGE = 7,        /* tt_encode_static only: len is above TT_STATIC_MAX_LEN              */
    TT_ERR_BAD_IDS = 8           /* tt_spans device status: unknown id, or the ids do not spell text_len bytes */
};

/* Patterns (benchmark configs; the paper names the two lineages in Sec. 4.1):
 *   TT_PATTERN_CL100K  contraction | [^\r\n\p{L}\p{N}]?\p{L}+ | \p{N}{1,3} | ' '?[^\s\p{L}\p{N}]+[\r\n]*
 *                      | \s*[\r\n]+ | \s+(?!\S) | \s+
 *   TT_PATTERN_O200K   case-aware word alternatives with an optional contraction suffix,
 *                      \p{N}{1,3}, ' '?[^\s\p{L}\p{N}]+[\r\n/]*, and the same whitespace rules.
 *   TT_PATTERN_CL100K_N1  TT_PATTERN_CL100K with \p{N} in place of \p{N}{1,3}: every digit is its own piece
 *                      (the "\p{N} single" front end of the paper's family table, App. A).
 *   TT_PATTERN_SPLIT3  three splitters in sequence (Sec. 4.1: each re-splits every piece of the stage before it, unmatched
 *                      spans survive as pieces): \p{N}{1,3} isolated, then [\p{Lm}\p{Lo}]+ isolated, then TT_PATTERN_CL100K
 *                      on every resulting span as a text of its own.  The paper prints no pattern of this family; this
 *                      composition is a stand-in with the same structure. */
enum { TT_PATTERN_CL100K = 0, TT_PATTERN_O200K = 1, TT_PATTERN_CL100K_N1 = 2, TT_PATTERN_SPLIT3 = 3 };

typedef struct tt_vocab tt_vocab;   /* opaque; immutable after load; owns its device tables */

/* One merge rule; its rank is its index in the array passed to tt_vocab_load. */
typedef struct { int32_t left, right, result; } tt_merge;

/*
 * tt_vocab_load -- build the device tables for one tokenizer (paper Sec. 4.2: merge ranks and
 * vocabulary entries are packed into GPU hash tables).
 *   merges    HOST, n_merges entries, copied.  rank = index.  `left`/`right` must each be a base id
 *             (a value of byte_map) or the `result` of a LOWER-ranked merge; pairs must be distinct;
 *             results must be distinct, non-negative and differ from every base id.
 *   byte_map  HOST, 256 entries: byte value -> base token id; must be injective and non-negative.
 *   pattern_id  TT_PATTERN_CL100K, TT_PATTERN_O200K, TT_PATTERN_CL100K_N1 or TT_PATTERN_SPLIT3.
 *   out       receives the handle (device tables live on the current CUDA device).
 * Limits: n_merges <= 262,144 - 256.  Synchronous (it waits for its own uploads).
 * Returns TT_OK, TT_ERR_ARG, TT_ERR_BAD_VOCAB or TT_ERR_CUDA; *out is NULL on failure.
 */
int tt_vocab_load(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256], int pattern_id,
                  tt_vocab** out);

/*
 * tt_vocab_load_ex -- tt_vocab_load with option flags.
 *   TT_VOCAB_IGNORE_MERGES  (paper Sec. 4.2: families configured with ignore_merges)  a piece whose bytes are,
 *             as a whole, the byte string of a vocabulary entry is encoded as that one entry without running
 *             the merge loop, whatever the merges would have made of it.  Where several entries spell the same
 *             bytes the base byte, else the lowest-ranked merge result, is taken.  All other pieces are merged
 *             as usual.  Entries of any length up to 4,096 bytes take part (those longer than 24 bytes through a
 *             second table); a vocabulary with a longer entry is refused with TT_ERR_BAD_VOCAB under this flag.
 * Everything else is as for tt_vocab_load (flags = 0 is the same call).  Unknown flag bits: TT_ERR_ARG.
 */
#define TT_VOCAB_IGNORE_MERGES 1u
int tt_vocab_load_ex(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256], int pattern_id,
                     unsigned flags, tt_vocab** out);

/* Frees the handle and its device tables.  NULL is allowed.  No encode using it may be in flight. */
void tt_vocab_free(tt_vocab* v);

/*
 * tt_vocab_table_entries -- number of vocabulary entries in the whole-piece table of `v` (paper Sec. 4.2 keeps
 * the vocabulary entries in a hash table on the GPU): the entries of at most 24 bytes whose own byte string
 * encodes to exactly that entry, i.e. the pieces that one table probe settles.  Host value, no device work.
 */
size_t tt_vocab_table_entries(const tt_vocab* v);

/*
 * tt_workspace_bytes -- DEVICE scratch size needed by an encode call over at most max_len text
 * bytes in at most max_docs documents (use 1 for tt_encode).  The caller allocates the scratch
 * (256-byte aligned) and may reuse it for any number of calls that do not overlap in time.  About 21.7 bytes per
 * text byte up to 4 MB of text, 28.3 beyond (texts that long use global work lists besides the per-tile ones); the
 * size never decreases as max_len grows, so scratch sized for the longest text serves every shorter one.
 */
size_t tt_workspace_bytes(const tt_vocab* v, size_t max_len, size_t max_docs);

/*
 * tt_encode -- tokenize one request (the cold full-request path, paper Sec. 4).
 *   text        DEVICE, len bytes of UTF-8 (len < 2^31).  Not modified.
 *   ids_out     DEVICE int32[ids_cap].  ids_cap >= len always suffices (a token covers >= 1 byte).
 *   count_out   DEVICE int64: number of tokens written (0 on a device-side error).
 *   status_out  DEVICE int32: TT_OK, TT_ERR_INVALID_UTF8, TT_ERR_CAPACITY or TT_ERR_INTERNAL_TIMEOUT.
 *   workspace   DEVICE scratch of at least tt_workspace_bytes(v, len, 1) bytes.
 * Asynchronous on `stream`.  len == 0 yields count 0, status TT_OK.
 * The call enqueues three kernels (for text of more than 4 MB four, behind a 128-byte memset; inside a stream
 * capture the memset is always there) and may be captured into a CUDA graph by the caller (paper Sec. 4.2: one
 * submission per request for a caller that reuses its buffers).
 */
int tt_encode(const tt_vocab* v, const uint8_t* text, size_t len, void* stream,
              int32_t* ids_out, size_t ids_cap, int64_t* count_out, int32_t* status_out,
              void* workspace, size_t workspace_bytes);

/*
 * tt_encode_batch -- tokenize n_docs independent documents in one call (paper Sec. 4.2:
 * multi-document batches concatenate inputs and cut runs at document boundaries).
 *   text         DEVICE, the documents concatenated; total_len = total bytes (HOST value, < 2^31).
 *   doc_off      DEVICE int64[n_docs+1], ascending byte offsets, doc_off[0]=0, doc_off[n_docs]=total_len.
 *   ids_out      DEVICE int32[ids_cap]: token IDs of all documents, in document order.
 *   ids_off_out  DEVICE int64[n_docs+1]: token offset of each document in ids_out; the last entry
 *                is the total count.
 *   status_out   DEVICE int32 as for tt_encode (one word for the whole batch; on error every
 *                ids_off_out entry is 0).
 * Every document is tokenized exactly as if it were encoded alone.  Asynchronous on `stream`.
 */
int tt_encode_batch(const tt_vocab* v, const uint8_t* text, size_t total_len, const int64_t* doc_off,
                    size_t n_docs, void* stream, int32_t* ids_out, size_t ids_cap, int64_t* ids_off_out,
                    int32_t* status_out, void* workspace, size_t workspace_bytes);

/*
 * tt_pretokenize -- the pre-tokenization half alone (paper Sec. 4.1; the paper checks piece
 * boundaries separately from IDs because ID-level agreement can hide a boundary fault).
 *   piece_off_out  DEVICE int32[piece_cap]: byte offset of every piece start, ascending, followed by one
 *                  closing entry piece_off_out[n_pieces] = len.  piece_cap must be at least len + 1 (a piece
 *                  has at least one byte, so that always suffices; a smaller capacity is refused with
 *                  TT_ERR_ARG before anything is enqueued).  With len == 0 nothing is written and any
 *                  capacity, also 0 with a null pointer, is accepted.
 *   n_pieces_out   DEVICE int64: number of pieces.
 * doc_off / n_docs as in tt_encode_batch, or doc_off = NULL and n_docs = 1 for one document.
 */
int tt_pretokenize(const tt_vocab* v, const uint8_t* text, size_t len, const int64_t* doc_off, size_t n_docs,
                   void* stream, int32_t* piece_off_out, size_t piece_cap, int64_t* n_pieces_out,
                   int32_t* status_out, void* workspace, size_t workspace_bytes);

/*
 * tt_spans -- byte and character spans of the tokens of an encoded text (paper App. E.3, span export:
 * the IDs gather per-token byte lengths, a cumulative sum yields byte offsets, and a second cumulative
 * sum over the non-continuation bytes lifts them to character offsets).
 *   ids, count      DEVICE: the IDs and their number, as tt_encode left them (count <= ids_cap).
 *   text_len        HOST value: byte length of the text the IDs were produced from (only checked).
 *   byte_off_out    DEVICE int32[ids_cap + 1]: token i covers text bytes [byte_off[i], byte_off[i+1]).
 *   char_off_out    DEVICE int32[ids_cap + 1]: char_off[i] = number of code points that start before
 *                   byte_off[i]; a token that begins inside a multi-byte character therefore starts at
 *                   the index of the next character.
 *   status_out      DEVICE int32: TT_OK, or TT_ERR_BAD_IDS if an id is not in the vocabulary or the
 *                   byte lengths do not add up to text_len (then only entry 0 of the outputs is written).
 *   workspace       DEVICE scratch of at least tt_spans_workspace_bytes(v, ids_cap) bytes, 256-byte aligned.
 * Asynchronous on `stream`; never reads the text.  Needs caller ids below 2^24 (else TT_ERR_ARG).
 */
size_t tt_spans_workspace_bytes(const tt_vocab* v, size_t ids_cap);
int tt_spans(const tt_vocab* v, const int32_t* ids, const int64_t* count, size_t ids_cap, size_t text_len,
             void* stream, int32_t* byte_off_out, int32_t* char_off_out, int32_t* status_out,
             void* workspace, size_t workspace_bytes);

/*
 * Added tokens (paper Sec. 4.3 / 4.4: added and special tokens are literal strings reserved as single ids; a
 * leftmost-longest literal pass extracts them before the tokenizer family handles the remaining segments).
 *   tt_vocab_add_literals  registers n literals once per vocabulary (HOST arrays, copied): literal i is
 *                          bytes[off[i] .. off[i+1]) (1..255 bytes, all distinct) with id ids[i] >= 0.
 *                          Returns TT_ERR_ARG for bad arguments or a second call.  tt_spans afterwards also
 *                          knows every literal whose id is below 2^24 and is not an id of the merge table.
 *   tt_encode_added        tt_encode with that pass in front: scanning left to right, at each byte the longest
 *                          literal that matches there is taken and the scan continues behind it; every taken literal
 *                          yields its id, and every stretch of text between literals is tokenized exactly as if it
 *                          were a text of its own.  Arguments, workspace and error behaviour as for tt_encode;
 *                          without registered literals it is tt_encode.
 */
int tt_vocab_add_literals(tt_vocab* v, const uint8_t* bytes, const uint32_t* off, const int32_t* ids, size_t n);
int tt_encode_added(const tt_vocab* v, const uint8_t* text, size_t len, void* stream,
                    int32_t* ids_out, size_t ids_cap, int64_t* count_out, int32_t* status_out,
                    void* workspace, size_t workspace_bytes);

/*
 * Sessions -- incremental repair on append (paper Sec. 3.3).  A session stores a text A and its tokenization as
 * records (byte position, id) in device memory.  tt_session_append(B) tokenizes only the last w characters of A
 * (w = 512 unless tt_session_set_window changed it) followed by B with the same kernels as tt_encode, looks for
 * the longest run of records on which the cached and the fresh sequence agree in position and id (the rightmost
 * of several), and admits it through the stable boundary check: at least two tokens, more characters than the
 * longest vocabulary entry, and a stable boundary at the start of one of its tokens (a character-class transition
 * after which the pieces do not depend on the text before it: whitespace, or punctuation other than a mark or an
 * apostrophe, after a letter or number; the first digit of a number; a letter after a number).  Cached records
 * are then kept up to the end of the run and fresh ones after it, in place.  If the check fails w doubles, at
 * most five times; after that, and whenever the window reaches the start of A, the whole text is tokenized.
 * The stored IDs always equal tt_encode of the whole text.
 *   tt_session_create   allocates the session's device buffers for up to max_bytes of text (about 40 bytes per
 *                       byte of capacity) on the current device; `v` must outlive the session.
 *   tt_session_append   text: HOST pointer, len bytes of valid UTF-8 (a complete string: it must not end inside
 *                       a character).  Synchronises `stream` (once per window tried).  info (HOST, may be NULL)
 *                       receives what happened.  An error (TT_ERR_INVALID_UTF8, TT_ERR_TOO_LARGE when the capacity
 *                       is exceeded, TT_ERR_CUDA) leaves the session unchanged.
 *   tt_session_view     DEVICE pointers to the IDs, to the byte offset of every token (count + 1 entries, the last
 *                       one the text length) and to the token count, plus the stored length in bytes; valid until
 *                       the next append or tt_session_free.
 *   tt_session_copy     copies the records into caller-owned DEVICE buffers, asynchronously on `stream`:
 *                       ids_out int32[ids_cap] (may be NULL), off_out int32[ids_cap + 1] (may be NULL), count_out
 *                       int64.  min(stored bytes, ids_cap) entries are copied (a token has at least one byte);
 *                       entries beyond the count are unspecified.
 * One session must not be used from two threads at once.
 */
typedef struct tt_session tt_session;
typedef struct {
    int32_t attempts;        /* windows tried (the full tokenization counts as one if it was the first try) */
    int32_t status;          /* TT_OK or the error that was returned                                        */
    int64_t window_chars;    /* window that was accepted, in characters; 0 = the whole text was tokenized    */
    int64_t window_start;    /* its first byte                                                               */
    int64_t run_tokens;      /* tokens in the matched run                                                    */
    int64_t splice_byte;     /* byte position from which fresh records were taken                            */
    int64_t n_tokens;        /* tokens now stored                                                            */
} tt_append_info;
int tt_session_create(const tt_vocab* v, size_t max_bytes, tt_session** out);
void tt_session_free(tt_session* s);
int tt_session_set_window(tt_session* s, uint32_t window_chars);
int tt_session_append(tt_session* s, const uint8_t* text, size_t len, void* stream, tt_append_info* info);
int tt_session_view(const tt_session* s, const int32_t** ids_dev, const int32_t** off_dev, const int64_t** count_dev,
                    size_t* len_bytes);
int tt_session_copy(const tt_session* s, int32_t* ids_out, size_t ids_cap, int32_t* off_out, int64_t* count_out,
                    void* stream);

/*
 * Shadow verification (paper Sec. 4.4): a background thread re-tokenizes a sample of the emitted sequences with a
 * reference engine and compares ids exactly; a mismatch is quarantined with a content hash for offline
 * reproduction; if the thread falls behind, samples are dropped and a visible counter is incremented.  Host only
 * (no GPU call); the reference engine is a callback of the caller.
 *   tt_verifier_create    reference(user, text, len, ids_out, ids_cap, count_out) must write the reference ids of
 *                         `text` (HOST buffers; ids_cap = len + 1) and return 0, or non-zero on failure (counted as
 *                         a mismatch).  sample_rate in [0, 1] (the paper serves with 0.05 and sweeps offline with 1);
 *                         queue_cap > 0 = samples that may wait; seed fixes which submissions are sampled.
 *   tt_verifier_submit    HOST text and ids of one emitted sequence (copied if sampled).  Returns 1 = queued,
 *                         0 = not sampled, 2 = sampled but dropped (queue full), -1 = bad arguments.  Never blocks
 *                         on the reference engine.
 *   tt_verifier_drain     waits until every queued sample has been checked.
 *   tt_verifier_get_stats counters so far.   tt_verifier_quarantined: mismatch `index` (0-based, at most 4,096 are
 *                         kept): 64-bit FNV-1a hash and length of its text, index of the first differing id (or
 *                         the shorter length; -2 if the reference engine failed).
 *   tt_verifier_free      finishes queued samples, stops the thread.
 */
typedef int (*tt_reference_fn)(void* user, const uint8_t* text, size_t len, int32_t* ids_out, size_t ids_cap,
                               int64_t* count_out);
typedef struct tt_verifier tt_verifier;
typedef struct { uint64_t submitted, sampled, checked, mismatches, dropped; } tt_verifier_stats;
int tt_verifier_create(tt_reference_fn reference, void* user, double sample_rate, size_t queue_cap, uint64_t seed,
                       tt_verifier** out);
int tt_verifier_submit(tt_verifier* q, const uint8_t* text, size_t len, const int32_t* ids, size_t n_ids);
void tt_verifier_drain(tt_verifier* q);
void tt_verifier_get_stats(tt_verifier* q, tt_verifier_stats* out);
int tt_verifier_quarantined(tt_verifier* q, size_t index, uint64_t* content_hash, uint64_t* len, int64_t* first_diff);
void tt_verifier_free(tt_verifier* q);

/*
 * tt_encode_timed -- diagnostic variant of tt_encode (same arguments and results) that records
 * CUDA events on `stream` between the kernels of the chain, waits for the last one and returns the
 * device time of each step in milliseconds: ms_out[0] the first kernel (tag + piece-start flags, per-tile
 * compaction and whole-piece lookups: K1+K2+K3+K4a), [1] merges of the pieces the lookups did not settle
 * (K4b), [2] token offsets and scatter (K5).  Synchronises; requires len > 0.  Used by the benchmark for the
 * per-kernel roofline; the event records perturb the chain slightly (the kernels are launched without
 * programmatic dependent launch here), so the sum exceeds the latency of a plain tt_encode call.
 */
int tt_encode_timed(const tt_vocab* v, const uint8_t* text, size_t len, void* stream, int32_t* ids_out,
                    size_t ids_cap, int64_t* count_out, int32_t* status_out, void* workspace,
                    size_t workspace_bytes, float ms_out[3]);

/*
 * tt_encode_host -- convenience wrapper for HOST buffers: copies `text` to the device, encodes,
 * delivers the IDs to `ids_out` and synchronises.  Allocates and caches its own device and pinned staging
 * buffers inside the handle's context (not thread-safe per vocab).  ids_out HOST int32[ids_cap];
 * *count_out HOST.  Page-locked caller buffers (cudaHostAlloc / cudaHostRegister, a pinned tensor) are used
 * directly: the first kernel reads `text` through the mapped pointer tile by tile (no copy in front of the chain; it
 * leaves a device copy for the later kernels), and the IDs are written by the scatter kernel through the mapped
 * pointer straight into `ids_out` (entries beyond the count are unspecified); pageable buffers are staged.
 * Returns the host code, or the device status if that is not TT_OK.
 */
int tt_encode_host(tt_vocab* v, const uint8_t* text, size_t len, int32_t* ids_out, size_t ids_cap,
                   int64_t* count_out);

/*
 * tt_encode_static -- tt_encode for callers that cannot provide scratch memory and must not allocate.
 * (The paper has no counterpart; this is a convenience of this library.)
 *
 * Some callers are not in a position to call cudaMalloc or to carve a workspace out of an allocator:
 * a plug-in running inside a serving process whose device memory is owned and budgeted by the host
 * framework, code on a latency-critical thread where an allocation could block behind the device's
 * other work, or a component that is handed only input and output buffers.  For them the scratch of
 * the kernel chain is a fixed array inside the library image: loading the library reserves
 * TT_STATIC_MAX_LEN * 28 + 65,536 bytes (about 7.1 MiB) on every GPU the process uses, until exit.
 *
 * Arguments and results are those of tt_encode without `workspace`; inputs and outputs are still
 * the caller's DEVICE buffers.  The call itself performs no cudaMalloc, cudaFree or other allocating
 * call.  Differences from tt_encode:
 *   - len above TT_STATIC_MAX_LEN (262,144 bytes) is refused with TT_ERR_TOO_LARGE; nothing is enqueued.
 *   - The first call on each device looks up the device address of the array (once per device, with
 *     that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, which still holds the previous call's data; the call
 *     clears the words that must start at zero.  Two calls whose kernels can overlap on the GPU
 *     (different streams, no ordering between them) race on it: order them on one stream or with events.
 */
#define TT_STATIC_MAX_LEN 262144u
int tt_encode_static(const tt_vocab* v, const uint8_t* text, size_t len, void* stream,
                     int32_t* ids_out, size_t ids_cap, int64_t* count_out, int32_t* status_out);

/*
 * Ranks and merge guards of token pairs as the merge kernels see them, computed on the HOST with no CUDA call
 * (for checks of the table construction).  Paper Sec. 4.2 merges, per round, the occurrences of the lowest
 * rank; the kernels also merge, in the same round, every pair that the sequential order is certain to merge:
 * a pair (x, y) of rank r with left neighbour u and right neighbour w such that r < cl(u, x) and
 * r <= cr(y, w), where
 *   cl(u, t) = lowest rank of a merge (X, t) whose left operand X has u on the right spine of its merge tree
 *              (X = u included),
 *   cr(t, w) = lowest rank of a merge (t, Y) whose right operand Y has w on the left spine of its merge tree.
 * left / right: n_pairs caller ids (HOST); out: 3 * n_pairs int64 (HOST): rank, cl, cr of each pair, -1 = none.
 * Returns TT_ERR_BAD_VOCAB / TT_ERR_ARG like tt_vocab_load.
 */
int tt_pair_info_host(const tt_merge* merges, size_t n_merges, const int32_t byte_map[256],
                      const int32_t* left, const int32_t* right, size_t n_pairs, int64_t* out);

/* Number of class-table entries (0x110000) copied to out (HOST uint8, one class code per code
 * point as the kernels see it): 0 other, 1 mark, 2 whitespace, 3 number, 4 lowercase letter,
 * 5 uppercase/titlecase letter, 6 caseless letter.  For exhaustive table checks. */
size_t tt_class_table(uint8_t* out, size_t cap);

/* Static, human-readable description of a code. */
const char* tt_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* TOKTIER_H */

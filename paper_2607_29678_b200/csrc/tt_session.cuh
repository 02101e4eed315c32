// Incremental repair on append (paper Sec. 3.3): kernels that compare the cached token records of a session
// with the records of a freshly tokenized window, apply the stable boundary check and splice in place.
//
// Records are (byte position, id).  The cached sequence is ids[0..ntok) with off[i] = first byte of token i
// and off[ntok] = length of the stored text; the fresh sequence covers the text from byte `ws` on (the last w
// characters of the stored text plus the appended text) with offsets relative to ws.  The longest run of
// fresh records that lie in the old part of the window and agree with a cached record in position, end and
// id is admitted if it has at least two tokens, covers more characters than the longest vocabulary entry
// and contains a stable boundary at the start of one of its tokens; then cached records are kept up to the
// end of the run and fresh records after it.
//
// Stable boundaries (all patterns; a subset of the positions that begin a piece whatever lies to their left,
// so the pieces from there on do not depend on the left context): a character c after a character q where
//   c is whitespace and q is a letter or a number;  c is a number and q is not;  c is a letter and q is a
//   number;  c is "other" (no mark, no apostrophe) and q is a letter or a number.
#pragma once
#include "tt_classify.cuh"

struct RepairDecision {
    int accept;                // 1: the run passed the check and the splice was applied
    int status;                // device status of the fresh tokenization (TT_OK or an error code)
    long long j0, j1;          // the run: fresh records [j0, j1)
    long long i1;              // cached records kept: [0, i1)
    long long new_ntok;        // tokens after the splice
    long long splice_byte;     // byte position where fresh records take over
};

struct RepairParams {
    int32_t* ids; int32_t* off; long long* ntok;                 // cached records (updated in place)
    const int32_t* fids; const int32_t* foff; const int32_t* fchar; const long long* fcount;   // fresh records
    const int32_t* fstatus; const int32_t* sstatus;              // device status of the fresh encode / span export
    const u8* text;                                              // the whole text (old + appended), device
    long long ws, old_len, new_len;
    const u8* cls; int cls_bytes;                                // class tables in global memory
    int max_tok_chars;
    u8* eq;                                                      // scratch: one flag per fresh record of the old part
    RepairDecision* dec;
};

__device__ __forceinline__ u32 session_class_at(const u8* text, long long p, const ClassTables& T, u32& cp_out) {
    const u32 b = text[p];
    u32 cp = b;
    if (b >= 0x80) {
        const int n = b >= 0xF0 ? 4 : b >= 0xE0 ? 3 : 2;
        cp = b & (0x7Fu >> n);
        for (int k = 1; k < n; k++) cp = (cp << 6) | (text[p + k] & 0x3F);
    }
    cp_out = cp;
    return cp < 0x80 ? (T.ascii[cp] & 7u) : tt_class_of(cp, T);
}

// Is byte position p (0 < p < len, the start of a token) a stable boundary?
__device__ __forceinline__ bool session_stable_boundary(const u8* text, long long p, long long len, const ClassTables& T) {
    if (p <= 0 || p >= len || (text[p] & 0xC0) == 0x80) return false;
    long long q = p - 1;
    for (int k = 0; k < 3 && q > 0 && (text[q] & 0xC0) == 0x80; k++) q--;
    u32 cp, cq;
    const u32 c = session_class_at(text, p, T, cp), pc = session_class_at(text, q, T, cq);
    const bool q_letter = pc == CC_LOWER || pc == CC_UPPER || pc == CC_CASELESS;
    const bool q_ln = q_letter || pc == CC_NUMBER;
    if (c == CC_SPACE) return q_ln;
    if (c == CC_NUMBER) return pc != CC_NUMBER;
    if (c == CC_LOWER || c == CC_UPPER || c == CC_CASELESS) return pc == CC_NUMBER;
    if (c == CC_OTHER) return cp != 0x27 && q_ln;
    return false;
}

// First index in [lo, hi) whose value is >= x (values ascending).
__device__ __forceinline__ long long session_lower_bound(const int32_t* a, long long lo, long long hi, long long x) {
    while (lo < hi) { const long long mid = (lo + hi) >> 1; if (a[mid] < x) lo = mid + 1; else hi = mid; }
    return lo;
}

// One CTA.  Writes the decision; the splice itself is done by k_repair_apply.
__global__ void __launch_bounds__(256)
k_repair_decide(const RepairParams P) {
    __shared__ long long s_jold, s_j0, s_j1;
    const int tid = threadIdx.x;
    ClassTables T;
    T.stage1 = P.cls; T.stage2 = P.cls + 0x1100; T.ascii = P.cls + P.cls_bytes - 128;
    const int status = *P.fstatus ? *P.fstatus : *P.sstatus;
    const long long nf = status ? 0 : *P.fcount, nA = *P.ntok;
    if (tid == 0) {
        // fresh records of the old part: those that end at or before old_len (ends ascend)
        long long lo = 0, hi = nf;
        while (lo < hi) { const long long mid = (lo + hi) >> 1; if (P.ws + P.foff[mid + 1] <= P.old_len) lo = mid + 1; else hi = mid; }
        s_jold = lo;
    }
    __syncthreads();
    const long long jold = s_jold;
    for (long long j = tid; j < jold; j += blockDim.x) {
        const long long p = P.ws + P.foff[j], e = P.ws + P.foff[j + 1];
        const long long i = session_lower_bound(P.off, 0, nA, p);
        P.eq[j] = (i < nA && P.off[i] == p && P.ids[i] == P.fids[j] && P.off[i + 1] == e) ? 1 : 0;
    }
    __syncthreads();
    if (tid == 0) {
        long long b0 = 0, b1 = 0;                       // longest run of agreement, the rightmost among equals
        for (long long j = 0; j < jold;) {
            if (!P.eq[j]) { j++; continue; }
            long long k = j;
            while (k < jold && P.eq[k]) k++;
            if (k - j >= b1 - b0) { b0 = j; b1 = k; }
            j = k;
        }
        s_j0 = b0; s_j1 = b1;
    }
    __syncthreads();
    const long long j0 = s_j0, j1 = s_j1;
    bool ok = (j1 - j0 >= 2) && (P.fchar[j1] - P.fchar[j0] > P.max_tok_chars);
    bool mine = false;
    if (ok) for (long long j = j0 + tid; j < j1 && !mine; j += blockDim.x) mine = session_stable_boundary(P.text, P.ws + P.foff[j], P.new_len, T);
    ok = __syncthreads_or(mine) && ok;
    if (tid == 0) {
        RepairDecision d;
        d.accept = ok ? 1 : 0; d.status = status; d.j0 = j0; d.j1 = j1; d.i1 = 0; d.new_ntok = nA; d.splice_byte = 0;
        if (ok) {
            d.i1 = session_lower_bound(P.off, 0, nA, P.ws + P.foff[j1 - 1]) + 1;
            d.new_ntok = d.i1 + (nf - j1);
            d.splice_byte = P.ws + P.foff[j1];
        }
        *P.dec = d;
    }
}

// Any grid.  Copies the fresh records behind the run over the cached ones and updates the count.
__global__ void __launch_bounds__(256)
k_repair_apply(const RepairParams P) {
    const RepairDecision d = *P.dec;
    if (!d.accept) return;
    const long long n = d.new_ntok - d.i1;
    for (long long k = (long long)blockIdx.x * blockDim.x + threadIdx.x; k < n; k += (long long)gridDim.x * blockDim.x) {
        P.ids[d.i1 + k] = P.fids[d.j1 + k];
        P.off[d.i1 + k] = (int32_t)(P.ws + P.foff[d.j1 + k]);
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) { P.off[d.new_ntok] = (int32_t)P.new_len; *P.ntok = d.new_ntok; }
}

// Span export: byte and character spans of the tokens of an encoded text.
//
// Paper App. E.3: the IDs gather per-token byte lengths, a cumulative sum yields byte offsets, and a
// second cumulative sum over the non-continuation text bytes lifts them to character offsets.  The
// tokens of a text concatenate to exactly its bytes, so the number of non-continuation bytes inside a
// token is a property of the token itself; both sums therefore run over per-token table values and the
// text is never read (its length only checks that the IDs belong to it).
#pragma once
#include "tt_common.cuh"
#include "tt_bpe.cuh"

constexpr int SPAN_THREADS = 1024;

struct SpanHeader {            // workspace header, zeroed at the start of every call
    u32 done;                  // CTAs that finished the block sums
    int status;
    u32 pad[30];
};

struct SpanParams {
    const int32_t* ids;
    const long long* count;    // DEVICE: number of ids
    unsigned long long ids_cap;
    unsigned long long text_len;
    const uint2* meta;         // per caller id: (byte length, non-continuation bytes); length 0 = unknown id
    u32 meta_n;
    SpanHeader* hdr;
    uint2* blk;                // per block of SPAN_THREADS tokens: (bytes, chars), then the exclusive prefix
    int32_t* byte_off;         // out [count + 1]
    int32_t* char_off;         // out [count + 1]
    int32_t* status_out;
};

__device__ __forceinline__ uint2 span_meta(const SpanParams& P, unsigned long long i, unsigned long long n, bool& bad) {
    uint2 m = make_uint2(0, 0);
    if (i < n) {
        const int32_t id = P.ids[i];
        if (id >= 0 && (u32)id < P.meta_n) m = P.meta[id];
        if (m.x == 0) bad = true;
    }
    return m;
}

// Pass 1: (bytes, chars) per block of tokens; the last CTA to finish scans the block sums.
__global__ void __launch_bounds__(SPAN_THREADS)
k_span_sums(const SpanParams P) {
    __shared__ u32 sc[40];
    __shared__ u32 s_islast;
    long long cnt = *P.count;
    if (cnt < 0 || (unsigned long long)cnt > P.ids_cap) { cnt = 0; if (threadIdx.x == 0) atomicMax(&P.hdr->status, 8); }
    const unsigned long long n = (unsigned long long)cnt;
    const unsigned long long nblk = (n + SPAN_THREADS - 1) / SPAN_THREADS;
    bool bad = false;
    for (unsigned long long b = blockIdx.x; b < nblk; b += gridDim.x) {
        const uint2 m = span_meta(P, b * SPAN_THREADS + threadIdx.x, n, bad);
        u32 t0, t1;
        cta_excl_sum_scan(m.x, sc, &t0);
        __syncthreads();
        cta_excl_sum_scan(m.y, sc, &t1);
        if (threadIdx.x == 0) P.blk[b] = make_uint2(t0, t1);
        __syncthreads();
    }
    if (bad) atomicMax(&P.hdr->status, 8 /* TT_ERR_BAD_IDS */);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) s_islast = (atomicAdd(&P.hdr->done, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!s_islast) return;
    __threadfence();
    unsigned long long c0 = 0, c1 = 0;
    for (unsigned long long b0 = 0; b0 < nblk; b0 += SPAN_THREADS) {
        const unsigned long long i = b0 + threadIdx.x;
        const uint2 x = i < nblk ? P.blk[i] : make_uint2(0, 0);
        u32 t0, t1;
        const u32 e0 = cta_excl_sum_scan(x.x, sc, &t0);
        __syncthreads();
        const u32 e1 = cta_excl_sum_scan(x.y, sc, &t1);
        if (i < nblk) P.blk[i] = make_uint2((u32)c0 + e0, (u32)c1 + e1);
        c0 += t0; c1 += t1;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        P.blk[nblk] = make_uint2((u32)c0, (u32)c1);
        if (c0 != P.text_len) atomicMax(&P.hdr->status, 8);     // the ids do not spell a text of this length
    }
}

// Pass 2: offsets of every token.
__global__ void __launch_bounds__(SPAN_THREADS)
k_span_write(const SpanParams P) {
    __shared__ u32 sc[40];
    long long cnt = *P.count;
    if (cnt < 0 || (unsigned long long)cnt > P.ids_cap) cnt = 0;
    const unsigned long long n = (unsigned long long)cnt;
    const unsigned long long nblk = (n + SPAN_THREADS - 1) / SPAN_THREADS;
    const int status = P.hdr->status;
    if (blockIdx.x == 0 && threadIdx.x == 0) {
        *P.status_out = status;
        if (status != 0 || n == 0) { P.byte_off[0] = 0; P.char_off[0] = 0; }
    }
    if (status != 0) return;
    bool bad = false;
    for (unsigned long long b = blockIdx.x; b < nblk; b += gridDim.x) {
        const unsigned long long i = b * SPAN_THREADS + threadIdx.x;
        const uint2 m = span_meta(P, i, n, bad);
        const uint2 base = P.blk[b];
        u32 t0, t1;
        const u32 e0 = cta_excl_sum_scan(m.x, sc, &t0);
        __syncthreads();
        const u32 e1 = cta_excl_sum_scan(m.y, sc, &t1);
        if (i < n) {
            P.byte_off[i] = (int32_t)(base.x + e0);
            P.char_off[i] = (int32_t)(base.y + e1);
            if (i == n - 1) { P.byte_off[n] = (int32_t)(base.x + e0 + m.x); P.char_off[n] = (int32_t)(base.y + e1 + m.y); }
        }
        __syncthreads();
    }
}

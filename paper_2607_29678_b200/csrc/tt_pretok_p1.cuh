// Pattern 1 (o200k-style) piece-start predicate.  (placeholder until the case-aware rules land)
#pragma once
#include "tt_pretok.cuh"

TT_HD u32 tt_eval_chunk_p1(const u16 (*sm)[TT_SLOTS], int slot, const u8* base, long long g0, long long hi,
                           const TileCarry& tc, bool have_tc, u32& need) {
    return tt_eval_chunk_p0(sm, slot, base, g0, hi, tc, have_tc, need);
}

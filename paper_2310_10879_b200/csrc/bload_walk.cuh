// Building blocks of the word-wise walks (the copy kernels for short runs, and the shifted copy of the consumer side): a
// warp walks a piece of the dense side of a call word by word; lane l takes the words l, l+32, ... and finds the run of
// each of its words in a window of 32 runs that the warp builds with one lane per run.  Device code only.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bload_internal.cuh"
#include "bload_warp_copy.cuh"

namespace bload {
namespace walk {

using wc::kFull;
using wc::warp_find_segment;

constexpr int kFar = 0x7fffffff;  // "beyond the warp's range"
__device__ __forceinline__ int clamp_far(int64_t v) { return v < 0 ? 0 : (v > (int64_t)kFar ? kFar : (int)v); }


// the run that holds byte lo0 of the call's dense side or, when lo0 lies in padding or in a filler block, the last run before it
__device__ __forceinline__ int first_run_at(const PlanView& pv, int n, int64_t block_begin, int64_t n_blocks, int64_t lo0,
                                            int64_t block_bytes, int fb, int lane)
{
    const int64_t q = lo0 / block_bytes, b = block_begin + q;
    if (b >= n_blocks) return n - 1;
    const int k0 = pv.block_seg_begin[b], k1 = pv.block_seg_begin[b + 1];
    const int64_t r0 = lo0 - q * block_bytes;
    return r0 < (int64_t)pv.block_fill[b] * fb ? warp_find_segment(pv.seg_start, k0, k1, (int)(r0 / fb), lane) : k1 - 1;
}
// window entry of run k for a walk along the dense side: where the run begins and ends there, relative to byte lo0 of the
// call's dense side and clamped to [0, kFar], and its place in the ragged store minus its (unclamped) begin.  A run ends
// where the next run of its block begins, or where the block's frames end.
__device__ __forceinline__ int4 dense_side_entry(const PlanView& pv, int n, int k, int64_t block_begin, int64_t block_bytes, int fb,
                                                 int64_t lo0)
{
    if (k >= n) return make_int4(kFar, kFar, 0, 0);
    const int blk = pv.seg_block[k], st = pv.seg_start[k];
    const int nst = k + 1 < n ? pv.seg_start[k + 1] : 0;  // a later run of the same block starts later
    const int e_slot = nst > st ? nst : pv.block_fill[blk];
    const int64_t d_flat = (blk - block_begin) * block_bytes + (int64_t)st * fb - lo0;
    const int64_t dl = pv.seg_src[k] * fb - d_flat;
    return make_int4(clamp_far(d_flat), clamp_far(d_flat + (int64_t)(e_slot - st) * fb), (int)(uint32_t)(uint64_t)dl,
                     (int)(uint32_t)((uint64_t)dl >> 32));
}

// A word of W bytes: the largest of 16, 8, 4, 2 and 1 that divides the frame size.
template <int W> struct WordOf { using type = uint32_t; };
template <> struct WordOf<1> { using type = unsigned char; };
template <> struct WordOf<2> { using type = unsigned short; };
template <> struct WordOf<8> { using type = uint2; };
template <> struct WordOf<16> { using type = uint4; };
template <int W>
__device__ __forceinline__ typename WordOf<W>::type load_word(const uint8_t* p)
{
    using T = typename WordOf<W>::type;
    return BLOAD_MAY_READ(p, W) ? __ldcs(reinterpret_cast<const T*>(p)) : T{};
}
template <int W>
__device__ __forceinline__ void store_word(uint8_t* p, typename WordOf<W>::type v)
{
    using T = typename WordOf<W>::type;
    if (BLOAD_MAY_WRITE(p, W)) __stcs(reinterpret_cast<T*>(p), v);
}
template <int W>
__device__ __forceinline__ typename WordOf<W>::type pad_word(uint32_t p4)
{
    using T = typename WordOf<W>::type;
    if constexpr (W == 16) return make_uint4(p4, p4, p4, p4);
    else if constexpr (W == 8) return make_uint2(p4, p4);
    else return (T)p4;
}

constexpr int kRangeChunkBytes = 16384;  // of the walked side per warp and turn, for calls that fill the machine
// The piece a warp takes per turn: 16 KB when that still gives every SM a few CTAs of 8 warps, else smaller (a multiple
// of 2 KB) so that a call of a few MB is spread over the machine instead of a handful of warps.
inline int walk_piece_bytes(int64_t total, int sm_count)
{
    const int64_t per_warp = total / ((int64_t)sm_count * 32);
    if (per_warp >= kRangeChunkBytes) return kRangeChunkBytes;
    const int64_t p = ((per_warp + 2047) / 2048) * 2048;
    return (int)(p < 2048 ? 2048 : p);
}

}  // namespace walk
}  // namespace bload

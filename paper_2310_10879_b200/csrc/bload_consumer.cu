// Consumer side of the start table (paper, Methods, second paragraph): a recurrent model hands
// information of frame t-1 to frame t and has to discard it wherever a new sequence starts inside a
// block.  These kernels use the plan's segment list for that, without per-slot metadata:
//   k11_carry_prev   prev[q, s, :] = dense[q, s-1, :] where a sequence continues at slot s, a fill byte
//                    elsewhere: one shifted, segmented memcpy over the whole batch (HBM bound);
//   k12_reset_state  one step of a slot-by-slot recurrence: rows of the carried state whose block does
//                    not continue a sequence at the given slot are re-initialised;
//   k14_repeat_last  the other padding the paper mentions: padding slots repeat the block's last frame;
//   k13_valid_sum    per-block sums of per-slot float values over frames only (padding masked out),
//                    in double precision and in a fixed order, plus their total.
#include "bload_internal.cuh"
#include "bload_warp_copy.cuh"
#include "bload_walk.cuh"

namespace bload {

namespace {

using namespace wc;
using namespace walk;

// Same decomposition as the pack kernel: the output is cut into sub-tiles of `sub_bytes`, a warp owns one.
// Inside a segment that occupies bytes [seg_b, seg_e) of its block, the first frame receives the fill byte and
// every later byte x receives dense[x - frame_bytes]; everything behind the last segment is fill.
__global__ void __launch_bounds__(256, 3) k11_carry_prev(PlanView pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                                                      int64_t block_count, const uint8_t* __restrict__ dense,
                                                      uint8_t* __restrict__ prev, int64_t sub_bytes, int64_t subs_per_block,
                                                      uint8_t fill_byte)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const uint8_t* s_limit = dense + block_count * block_bytes;

    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_block;
        const int64_t lo = (item - q * subs_per_block) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, block_bytes);
        const int64_t b = block_begin + q;
        const int64_t dense_off = q * block_bytes;
        int64_t cur = lo;
        if (b < n_blocks) {
            const int k0 = pv.block_seg_begin[b], k1 = pv.block_seg_begin[b + 1];
            const int fill = pv.block_fill[b];
            if (cur < (int64_t)fill * frame_bytes) {
                int k = warp_find_segment(pv.seg_start, k0, k1, (int)(cur / frame_bytes), lane);
                int kw = k;  // lanes hold the start slots of segments kw .. kw+31
                int w_st = (kw + lane < k1) ? pv.seg_start[kw + lane] : fill;
                while (cur < hi && k < k1) {
                    if (k - kw == 31) {
                        kw = k;
                        w_st = (kw + lane < k1) ? pv.seg_start[kw + lane] : fill;
                    }
                    const int st = __shfl_sync(kFull, w_st, k - kw);
                    const int nx = __shfl_sync(kFull, w_st, k - kw + 1);
                    const int64_t first_e = min(((int64_t)st + 1) * frame_bytes, hi);  // end of the first frame
                    const int64_t seg_e = min((int64_t)nx * frame_bytes, hi);
                    if (cur < first_e) {
                        warp_fill(prev + dense_off + cur, first_e - cur, fill_byte, lane);
                        cur = first_e;
                    }
                    if (cur < seg_e) {
                        warp_copy<true>(prev + dense_off + cur, dense + dense_off + cur - frame_bytes, seg_e - cur, s_limit, lane);
                        cur = seg_e;
                    }
                    ++k;
                }
            }
        }
        if (cur < hi) warp_fill(prev + dense_off + cur, hi - cur, fill_byte, lane);
    }
}

// The same result for short runs (many segments per sub-tile).  Inside the occupied part of a block, prev is the
// dense input moved up by one frame -- the segments only matter at their first frames.  So a warp copies the
// occupied part of its sub-tile as ONE shifted run, whatever the segments are (no per-segment alignment work, the
// bytes in flight of a long run), fills the padding behind it, and then overwrites the first frame of every segment
// that starts inside the sub-tile with the fill byte: one lane per segment for small frames, the whole warp per
// segment for larger ones.  The patches are ordered after the copy's stores by a warp barrier.
__global__ void __launch_bounds__(256, 3) k11_carry_shift(PlanView pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                                                       int64_t block_count, const uint8_t* __restrict__ dense,
                                                       uint8_t* __restrict__ prev, int64_t sub_bytes, int64_t subs_per_block,
                                                       uint8_t fill_byte)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const uint8_t* s_limit = dense + block_count * block_bytes;
    const uint32_t f4 = 0x01010101u * fill_byte;

    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_block;
        const int64_t lo = (item - q * subs_per_block) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, block_bytes);
        const int64_t b = block_begin + q;
        uint8_t* out = prev + q * block_bytes;
        int k0 = 0, k1 = 0;
        int64_t valid_e = lo;  // end of the occupied part of [lo, hi)
        if (b < n_blocks) {
            k0 = pv.block_seg_begin[b]; k1 = pv.block_seg_begin[b + 1];
            valid_e = max(lo, min(hi, (int64_t)pv.block_fill[b] * frame_bytes));
        }
        const int64_t c0 = max(lo, frame_bytes);  // slot 0 has no slot before it (and always starts a segment)
        if (c0 < valid_e) warp_copy<true>(out + c0, dense + q * block_bytes + c0 - frame_bytes, valid_e - c0, s_limit, lane);
        if (valid_e < hi) warp_fill(out + valid_e, hi - valid_e, fill_byte, lane);
        if (lo >= valid_e) continue;
        __syncwarp();
        // first frames of the segments that reach into [lo, valid_e): segment ka holds the slot of byte lo
        const int ka = warp_find_segment(pv.seg_start, k0, k1, (int)(lo / frame_bytes), lane);
        for (int base = ka; base < k1; base += 32) {
            const int kk = base + lane;
            int64_t a = valid_e, e = valid_e;  // this lane's patch [a, e), empty by default
            if (kk < k1) {
                const int64_t fa = (int64_t)pv.seg_start[kk] * frame_bytes;
                a = min(max(fa, lo), valid_e);
                e = min(max(fa + frame_bytes, lo), valid_e);
            }
            if (frame_bytes <= 64) {
                if (((a | e | reinterpret_cast<uintptr_t>(out)) & 3) == 0)
                    for (int64_t x = a; x < e; x += 4) put_word(out + x, f4);
                else
                    for (int64_t x = a; x < e; ++x) put_byte(out + x, fill_byte);
            } else {
                const unsigned live = __ballot_sync(kFull, a < e);
                for (unsigned m = live; m; m &= m - 1) {
                    const int src_lane = __ffs(m) - 1;
                    const int64_t pa = __shfl_sync(kFull, a, src_lane), pe = __shfl_sync(kFull, e, src_lane);
                    warp_fill(out + pa, pe - pa, fill_byte, lane);
                }
            }
            // segments are in slot order: once one starts at or behind the end of the range, the rest do too
            const bool beyond = kk >= k1 || (int64_t)pv.seg_start[kk] * frame_bytes >= valid_e;
            if (__any_sync(kFull, beyond)) break;
        }
    }
}

// A warp owns `sub_bytes` of one row of the state.  It decides from the plan whether a sequence continues at
// `slot` of the row's block (then the row is left alone) and otherwise writes the initial state over its part.
__global__ void __launch_bounds__(256) k12_reset_state(PlanView pv, int64_t block_begin, int64_t block_count, int32_t slot,
                                                       uint8_t* __restrict__ state, int64_t state_bytes,
                                                       const uint8_t* __restrict__ init, int64_t sub_bytes,
                                                       int64_t subs_per_row)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_row;
    const int64_t n_blocks = pv.hdr->n_blocks;
    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_row;
        const int64_t lo = (item - q * subs_per_row) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, state_bytes);
        const int64_t b = block_begin + q;
        bool continues = false;
        if (b < n_blocks && slot < pv.block_fill[b]) {
            const int k = warp_find_segment(pv.seg_start, pv.block_seg_begin[b], pv.block_seg_begin[b + 1], slot, lane);
            continues = pv.seg_start[k] != slot;
        }
        if (continues) continue;
        uint8_t* d = state + q * state_bytes + lo;
        if (init) warp_copy<true>(d, init + lo, hi - lo, init + state_bytes, lane);
        else warp_fill(d, hi - lo, 0, lane);
    }
}

// Repeat-last padding, applied after the pack kernel has written the blocks: a warp owns a sub-tile of the dense
// side and overwrites the part of it that lies in the padding of its block with copies of the block's last frame.
__global__ void __launch_bounds__(256) k14_repeat_last(PlanView pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                                                       int64_t block_count, uint8_t* __restrict__ dense, int64_t sub_bytes,
                                                       int64_t subs_per_block)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_block;
        const int64_t b = block_begin + q;
        if (b >= n_blocks) continue;  // a filler block has no frame to repeat
        const int64_t pad_lo = (int64_t)pv.block_fill[b] * frame_bytes;
        const int64_t lo = (item - q * subs_per_block) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, block_bytes);
        int64_t cur = max(lo, pad_lo);
        if (cur >= hi || pad_lo == 0) continue;
        uint8_t* row = dense + q * block_bytes;
        const uint8_t* last = row + pad_lo - frame_bytes;
        int64_t fo = cur % frame_bytes;  // offset inside the frame being written
        while (cur < hi) {
            const int64_t len = min(frame_bytes - fo, hi - cur);
            warp_copy<true>(row + cur, last + fo, len, row + pad_lo, lane);
            cur += len;
            fo = 0;
        }
    }
}

// The same for small frames (below 512 bytes), where a copy per padding frame costs more than the frame: the padding
// part of the sub-tile is written word by word, lane l the words l, l+32, ...; a word at byte x of the padding comes from
// byte x mod frame_bytes of the last frame.  A word is the largest of 16, 8, 4, 2 and 1 bytes that divides the frame.
template <int W>
__global__ void __launch_bounds__(256) k14_repeat_last_words(PlanView pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                                                             int64_t block_count, uint8_t* __restrict__ dense, int64_t sub_bytes,
                                                             int64_t subs_per_block)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int fb = (int)frame_bytes;
    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_block;
        const int64_t b = block_begin + q;
        if (b >= n_blocks) continue;  // a filler block has no frame to repeat
        const int64_t pad_lo = (int64_t)pv.block_fill[b] * frame_bytes;
        const int64_t lo = (item - q * subs_per_block) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, block_bytes);
        const int64_t cur = max(lo, pad_lo);
        if (cur >= hi || pad_lo == 0) continue;
        uint8_t* row = dense + q * block_bytes;
        const uint8_t* last = row + pad_lo - frame_bytes;
        // (pad_lo, lo and frame_bytes are multiples of W: so are cur and every offset below)
        int off = (int)((cur - pad_lo + (int64_t)W * lane) % fb);  // offset of this lane's first word inside the frame
        const int step = (32 * W) % fb;
        for (int64_t x = cur + (int64_t)W * lane; x < hi; x += 32 * W) {
            store_word<W>(row + x, load_word<W>(last + off));
            off += step;
            if (off >= fb) off -= fb;
        }
    }
}
using RepeatWordsKernel = void (*)(PlanView, int32_t, int64_t, int64_t, int64_t, uint8_t*, int64_t, int64_t);
inline RepeatWordsKernel repeat_words_kernel_for(int64_t frame_bytes)
{
    return frame_bytes % 16 == 0 ? k14_repeat_last_words<16> : frame_bytes % 8 == 0 ? k14_repeat_last_words<8>
           : frame_bytes % 4 == 0 ? k14_repeat_last_words<4> : frame_bytes % 2 == 0 ? k14_repeat_last_words<2> : k14_repeat_last_words<1>;
}

constexpr int kSumThreads = 256;

// Fixed-order sum of one double per thread over a CTA of kSumThreads threads; the result is valid in thread 0.
__device__ __forceinline__ double cta_sum(double v, double* sh)
{
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) v += __shfl_down_sync(kFull, v, d);
    if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
    __syncthreads();
    double t = 0.0;
    if (threadIdx.x == 0)
        for (int w = 0; w < kSumThreads / 32; ++w) t += sh[w];
    __syncthreads();
    return t;
}

// One CTA per block: the frames of a block are its first block_fill slots, so the mask needs no segment search.
__global__ void __launch_bounds__(kSumThreads) k13_valid_sum(PlanView pv, int32_t t_block, int64_t block_begin,
                                                             const float* __restrict__ values,
                                                             double* __restrict__ block_sum)
{
    __shared__ double sh[kSumThreads / 32];
    const int64_t q = blockIdx.x;
    const int64_t b = block_begin + q;
    const int fill = b < pv.hdr->n_blocks ? pv.block_fill[b] : 0;
    const float* row = values + q * (int64_t)t_block;
    double acc = 0.0;
    if ((reinterpret_cast<uintptr_t>(row) & 15u) == 0) {
        const int nv = fill >> 2;
        const float4* r4 = reinterpret_cast<const float4*>(row);
        int i = threadIdx.x;
        for (; i + 3 * kSumThreads < nv; i += 4 * kSumThreads) {  // four loads in flight per thread
            float4 v[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) v[u] = __ldcs(r4 + i + u * kSumThreads);
#pragma unroll
            for (int u = 0; u < 4; ++u) acc += ((double)v[u].x + (double)v[u].y) + ((double)v[u].z + (double)v[u].w);
        }
        for (; i < nv; i += kSumThreads) {
            const float4 v = __ldcs(r4 + i);
            acc += ((double)v.x + (double)v.y) + ((double)v.z + (double)v.w);
        }
        for (int i = (nv << 2) + threadIdx.x; i < fill; i += kSumThreads) acc += (double)row[i];
    } else {
        for (int i = threadIdx.x; i < fill; i += kSumThreads) acc += (double)row[i];
    }
    const double t = cta_sum(acc, sh);
    if (threadIdx.x == 0) block_sum[q] = t;
}

// Short blocks: a warp per block (eight blocks per CTA), the same masked sum in a fixed order (lane-strided partial sums,
// then the shuffle tree).  With one CTA per block half a million blocks of 94 slots took 0.9 ms.
__global__ void __launch_bounds__(kSumThreads) k13_valid_sum_short(PlanView pv, int32_t t_block, int64_t block_begin,
                                                                   int64_t block_count, const float* __restrict__ values,
                                                                   double* __restrict__ block_sum)
{
    const int lane = threadIdx.x & 31;
    const int64_t n_blocks = pv.hdr->n_blocks;
    for (int64_t q = (int64_t)blockIdx.x * (kSumThreads / 32) + (threadIdx.x >> 5); q < block_count;
         q += (int64_t)gridDim.x * (kSumThreads / 32)) {
        const int64_t b = block_begin + q;
        const int fill = b < n_blocks ? pv.block_fill[b] : 0;
        const float* row = values + q * (int64_t)t_block;
        double acc = 0.0;
        for (int i = lane; i < fill; i += 32) acc += (double)__ldcs(row + i);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_down_sync(kFull, acc, d);
        if (lane == 0) block_sum[q] = acc;
    }
}

// total[0] = sum of the block sums, total[1] = number of frames in the range; one CTA, fixed order.
__global__ void __launch_bounds__(kSumThreads) k13_total(PlanView pv, int64_t block_begin, int64_t block_count,
                                                         const double* __restrict__ block_sum, double* __restrict__ total)
{
    __shared__ double sh[kSumThreads / 32];
    const int64_t n_blocks = pv.hdr->n_blocks;
    double s = 0.0, c = 0.0;
    int64_t q = threadIdx.x;
    for (; q + 3 * kSumThreads < block_count; q += 4 * kSumThreads) {  // four loads of each kind in flight per thread
        double v[4];
        int f[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            v[u] = block_sum[q + u * kSumThreads];
            f[u] = block_begin + q + u * kSumThreads < n_blocks ? pv.block_fill[block_begin + q + u * kSumThreads] : 0;
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) { s += v[u]; c += (double)f[u]; }
    }
    for (; q < block_count; q += kSumThreads) {
        s += block_sum[q];
        if (block_begin + q < n_blocks) c += (double)pv.block_fill[block_begin + q];
    }
    const double ts = cta_sum(s, sh);
    const double tc = cta_sum(c, sh);
    if (threadIdx.x == 0) { total[0] = ts; total[1] = tc; }
}

// The shifted copy as a word-wise walk along the dense side (see bload_walk.cuh), for short runs and small blocks: lane l
// takes the words l, l+32, ... of 16 KB of the output and finds the run of each of its words in a window of 32 runs.  A
// word of a run's first frame, of padding or of a filler block receives the fill byte, every other word x receives
// dense[x - frame_bytes]: loads and stores of a warp are contiguous.  A window entry: {begin of the next run, end of this
// run, begin of this run}, relative to the first byte of the warp's piece.
template <int W>
__global__ void __launch_bounds__(256) k23_carry_walk(PlanView pv, int32_t n, int32_t t_block, int64_t frame_bytes,
                                                      int64_t block_begin, const uint8_t* __restrict__ dense,
                                                      uint8_t* __restrict__ prev, int64_t total, uint8_t fill, int32_t piece)
{
    __shared__ int4 windows[8][32];
    constexpr int U = W == 16 ? 4 : 8;  // words in flight per lane
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int4* win = windows[warp];
    const int fb = (int)frame_bytes;
    const int64_t block_bytes = (int64_t)t_block * fb;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int64_t chunks = (total + piece - 1) / piece;
    const uint32_t f4 = 0x01010101u * fill;
    for (int64_t c = (int64_t)blockIdx.x * 8 + warp; c < chunks; c += (int64_t)gridDim.x * 8) {
        const int64_t lo0 = c * (int64_t)piece;  // positions below are relative to this byte of the call's dense side
        const int p_end = (int)min((int64_t)piece, total - lo0);
        int kw = first_run_at(pv, n, block_begin, n_blocks, lo0, block_bytes, fb, lane);
        int r = 0, e = 0, b = 0, dn = 0, d_last = 0;
        auto load_window = [&]() {  // one lane per run
            const int k = kw + lane;
            int4 w = make_int4(kFar, kFar, 0, 0);
            if (k < n) {
                const int blk = pv.seg_block[k], st = pv.seg_start[k];
                const int nst = k + 1 < n ? pv.seg_start[k + 1] : 0;  // a later run of the same block starts later
                const int e_slot = nst > st ? nst : pv.block_fill[blk];
                const int64_t d_flat = (blk - block_begin) * block_bytes + (int64_t)st * fb - lo0;
                // (a run that began before this piece began inside the same block: more than -2^30; one that lies before
                // the call's blocks is clamped, its end is 0 and its begin is never looked at)
                const int64_t b_true = d_flat < -(1LL << 30) ? -(1LL << 30) : d_flat;
                w = make_int4(clamp_far(d_flat), clamp_far(d_flat + (int64_t)(e_slot - st) * fb), b_true > (int64_t)kFar ? kFar : (int)b_true, 0);
            }
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, 0);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; e = w0.y; b = w0.z;
        };
        load_window();
        const uint8_t* src = dense + lo0 - fb;  // the word at position q comes from position q - frame_bytes
        uint8_t* out = prev + lo0;
        int done = 0;
        while (done < p_end) {  // ends: a turn reaches p_end or moves the window on by 31 runs that begin ever later
            const int limit = min(p_end, d_last);
            for (int p = done + W * lane; p < limit; p += 32 * W * U) {
                bool carried[U];
                typename WordOf<W>::type v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = p + u * 32 * W;
                    carried[u] = false;
                    if (q < limit) {
                        while (q >= dn) {  // (q < limit <= begin of the window's last entry, so r stays below 31)
                            ++r;
                            const int4 w = win[r];
                            dn = w.x; e = w.y; b = w.z;
                        }
                        carried[u] = q < e && q - b >= fb;
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) v[u] = carried[u] ? load_word<W>(src + p + u * 32 * W) : pad_word<W>(f4);
#pragma unroll
                for (int u = 0; u < U; ++u) if (p + u * 32 * W < limit) store_word<W>(out + p + u * 32 * W, v[u]);
            }
            done = limit;
            if (limit == d_last) { kw += 31; load_window(); }
        }
    }
}
using CarryWalkKernel = void (*)(PlanView, int32_t, int32_t, int64_t, int64_t, const uint8_t*, uint8_t*, int64_t, uint8_t, int32_t);
inline CarryWalkKernel carry_walk_kernel_for(int64_t frame_bytes)
{
    return frame_bytes % 16 == 0 ? k23_carry_walk<16> : frame_bytes % 8 == 0 ? k23_carry_walk<8>
           : frame_bytes % 4 == 0 ? k23_carry_walk<4> : frame_bytes % 2 == 0 ? k23_carry_walk<2> : k23_carry_walk<1>;
}
// When the walk replaces the sub-tile kernels.  Measured on B200 (TB/s, walk against k11_carry_shift; clips = blocks of 94
// frames in runs of 22): 8-byte frames of clips 4.87 against 1.33, 16-byte 5.85 against 2.41, 64-byte 6.21 against 4.31,
// 256-byte 6.36 against 5.43, 6-byte 2.72 against 1.07 (the sub-tile kernels take a block per warp at least: 752 bytes);
// blocks of 10,000 frames in runs of 58: 16-byte frames 6.25 against 5.47, 64-byte 6.29 against 6.11, 256-byte (15 KB
// runs) 6.41 against 6.51, 8-byte 5.86 against 5.90, 4-byte 4.59 against 5.33, 6-byte 3.29 against 5.19; token lengths:
// 8- and 16-byte frames level, 4-byte 5.91 against 6.26, 64-byte and larger 2-3 % behind.
inline bool carry_walks(int64_t frame_bytes, int64_t mean_run, int64_t block_bytes)
{
    if (block_bytes <= 1024 || (block_bytes <= 4096 && frame_bytes % 4 == 0)) return true;  // (1-byte frames in blocks of 4 KB: 2.0 against 5.1)
    return frame_bytes % 8 == 0 && (mean_run <= 8192 || block_bytes <= 32768) && mean_run <= 16384;
}

unsigned grid_for_items(int64_t items)
{
    const int64_t want = (items + 7) / 8;  // CTAs of 8 warps, one item per warp
    return (unsigned)(want < 0x7fffffffLL ? want : 0x7fffffffLL);
}

}  // namespace

cudaError_t launch_carry_prev(const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                              int64_t block_count, const uint8_t* dense, uint8_t* prev, uint8_t fill_byte, cudaStream_t st,
                              int64_t n, int64_t sum_t)
{
    if (block_count == 0) return cudaSuccess;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t sub = 16384;
    const int64_t spb = (block_bytes + sub - 1) / sub;
    count_launches(1);
    BLOAD_DBG_EXPECT(st, dbg::kCarry, {{dense, (size_t)(block_count * block_bytes)}}, {{prev, (size_t)(block_count * block_bytes)}});
    if (n > 0 && n < 0x7fffff00LL && block_bytes < (1LL << 30) && carry_walks(frame_bytes, sum_t * frame_bytes / n, block_bytes)) {
        const int64_t total = block_count * block_bytes;
        const int piece = walk_piece_bytes(total, device_info().sm_count);
        const int64_t want = ((total + piece - 1) / piece + 7) / 8;
        const int64_t cap = (int64_t)device_info().sm_count * 32;
        note_copy_kernel(kCallCarryPrev, "k23_carry_walk");
        carry_walk_kernel_for(frame_bytes)<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(pv, (int32_t)n, t_block, frame_bytes, block_begin,
                                                                                                dense, prev, total, fill_byte, piece);
        return cudaPeekAtLastError();
    }
    // short runs (many segments per sub-tile): one shifted copy per sub-tile and patches at the segment starts
    if (n > 0 && sum_t * frame_bytes / n <= 16384) {
        note_copy_kernel(kCallCarryPrev, "k11_carry_shift");
        k11_carry_shift<<<grid_for_items(block_count * spb), 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count,
                                                                          dense, prev, sub, spb, fill_byte);
        return cudaPeekAtLastError();
    }
    note_copy_kernel(kCallCarryPrev, "k11_carry_prev");
    k11_carry_prev<<<grid_for_items(block_count * spb), 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count,
                                                                     dense, prev, sub, spb, fill_byte);
    return cudaPeekAtLastError();
}

cudaError_t launch_reset_state(const PlanView& pv, int64_t block_begin, int64_t block_count, int32_t slot, uint8_t* state,
                               int64_t state_bytes, const uint8_t* init, cudaStream_t st)
{
    if (block_count == 0) return cudaSuccess;
    const int64_t sub = 16384;
    const int64_t spr = (state_bytes + sub - 1) / sub;
    count_launches(1);
    BLOAD_DBG_EXPECT(st, dbg::kResetState, {{init, (size_t)state_bytes}}, {{state, (size_t)(block_count * state_bytes)}});
    k12_reset_state<<<grid_for_items(block_count * spr), 256, 0, st>>>(pv, block_begin, block_count, slot, state, state_bytes,
                                                                      init, sub, spr);
    return cudaPeekAtLastError();
}

cudaError_t launch_repeat_last(const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                               int64_t block_count, uint8_t* dense, cudaStream_t st)
{
    if (block_count == 0) return cudaSuccess;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t sub = 16384;
    const int64_t spb = (block_bytes + sub - 1) / sub;
    count_launches(1);
    BLOAD_DBG_EXPECT(st, dbg::kRepeatLast, {{dense, (size_t)(block_count * block_bytes)}}, {{dense, (size_t)(block_count * block_bytes)}});
    if (frame_bytes < 512)
        repeat_words_kernel_for(frame_bytes)<<<grid_for_items(block_count * spb), 256, 0, st>>>(pv, t_block, frame_bytes, block_begin,
                                                                                                block_count, dense, sub, spb);
    else
        k14_repeat_last<<<grid_for_items(block_count * spb), 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count,
                                                                          dense, sub, spb);
    return cudaPeekAtLastError();
}

cudaError_t launch_valid_sum(const PlanView& pv, int32_t t_block, int64_t block_begin, int64_t block_count,
                             const float* values, double* block_sum, double* total, cudaStream_t st)
{
    if (block_count == 0) return cudaSuccess;
    count_launches(total ? 2 : 1);
    if (t_block <= 1024) {  // a warp per block
        const int64_t want = (block_count + kSumThreads / 32 - 1) / (kSumThreads / 32), cap = (int64_t)device_info().sm_count * 64;
        k13_valid_sum_short<<<(unsigned)(want < cap ? want : cap), kSumThreads, 0, st>>>(pv, t_block, block_begin, block_count, values,
                                                                                       block_sum);
    } else {
        k13_valid_sum<<<(unsigned)block_count, kSumThreads, 0, st>>>(pv, t_block, block_begin, values, block_sum);
    }
    if (total) k13_total<<<1, kSumThreads, 0, st>>>(pv, block_begin, block_count, block_sum, total);
    return cudaPeekAtLastError();
}

}  // namespace bload

// Frames whose size differs from sample to sample (paper, Problem Statement: every sample S_i has its own
// H, W and T).  Sequence i holds T_i frames of F_i bytes back to back; a slot of a block has room for the
// largest frame, and a smaller frame sits at the start of its slot, followed by padding.
//   k15_var_offsets  byte offset of every sequence in such a store (exclusive scan of T_i * F_i), with the
//                    largest frame size and the first invalid size;
//   k16_copy_var     pack / unpack with per-sequence frame sizes, optionally as images of rows x row bytes on a
//                    canvas: the decomposition of the fixed-size copy kernel (a warp owns a sub-tile of the dense
//                    side), walking the canvas rows inside each segment.
#include "bload_internal.cuh"
#include "bload_warp_copy.cuh"

namespace bload {

namespace {

using namespace wc;

constexpr int kScanThreads = 1024;

// One CTA walks the sequences in chunks of kScanThreads with a running carry.  out[0..n) = first byte of each
// sequence, out[n] = total bytes, out[n+1] = largest frame size, out[n+2] = first i with F_i < 1 (or -1).
__global__ void __launch_bounds__(kScanThreads) k15_var_offsets(const int32_t* __restrict__ lengths,
                                                                const int32_t* __restrict__ rows /*null: one row*/,
                                                                const int32_t* __restrict__ frame_bytes, int64_t n,
                                                                int64_t* __restrict__ out, int64_t* __restrict__ max_rows)
{
    __shared__ int64_t warp_sum[kScanThreads / 32];
    __shared__ int64_t carry_sh;
    __shared__ int max_sh, max_rows_sh;
    __shared__ unsigned long long bad_sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { carry_sh = 0; max_sh = 0; max_rows_sh = 0; bad_sh = ~0ULL; }
    __syncthreads();
    int my_max = 0, my_rows = 0;
    for (int64_t base = 0; base < n; base += kScanThreads) {
        const int64_t i = base + threadIdx.x;
        int64_t v = 0;
        if (i < n) {
            const int f = frame_bytes[i];
            const int h = rows ? rows[i] : 1;
            if (f < 1 || h < 1) atomicMin(&bad_sh, (unsigned long long)i);
            my_max = max(my_max, f);
            my_rows = max(my_rows, h);
            v = (int64_t)lengths[i] * (int64_t)max(h, 0) * (int64_t)max(f, 0);
        }
        int64_t incl = v;  // inclusive scan inside the warp
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int64_t up = __shfl_up_sync(kFull, incl, d);
            if (lane >= d) incl += up;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            int64_t w = warp_sum[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const int64_t up = __shfl_up_sync(kFull, w, d);
                if (lane >= d) w += up;
            }
            warp_sum[lane] = w;  // inclusive over warps
        }
        __syncthreads();
        const int64_t carry = carry_sh;
        const int64_t before = carry + (warp ? warp_sum[warp - 1] : 0) + (incl - v);
        if (i < n) out[i] = before;
        __syncthreads();
        if (threadIdx.x == kScanThreads - 1) carry_sh = carry + warp_sum[kScanThreads / 32 - 1];
        __syncthreads();
    }
    atomicMax(&max_sh, my_max);
    atomicMax(&max_rows_sh, my_rows);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (max_rows) *max_rows = max_rows_sh;
        out[n] = carry_sh;
        out[n + 1] = max_sh;
        out[n + 2] = bad_sh == ~0ULL ? -1 : (int64_t)bad_sh;
    }
}

// Division of a 32-bit unsigned number by a divisor fixed at launch: a multiply-high and two shifts
// (Granlund and Montgomery, "Division by invariant integers using multiplication", PLDI 1994).
struct FastDiv { uint32_t mul, sh1, sh2, d; };
__device__ __forceinline__ uint32_t fast_div(uint32_t n, const FastDiv& f)
{
    const uint32_t t = __umulhi(f.mul, n);
    return (t + ((n - t) >> f.sh1)) >> f.sh2;
}

// Frames are images of `rows` rows of `frame_bytes` (row) bytes; a slot is a canvas of rows_max rows of row_stride
// bytes and an image sits in its top left corner (one row per frame and rows_max == 1 give the plain
// per-sequence frame size).  The dense side is walked row by row of the canvases ("sub-slots" of row_stride
// bytes).  Row counts and row sizes are clamped to the canvas on the device, so a caller that breaks the documented
// precondition gets truncated images but never an access outside the buffers.
// Four CTAs per SM: with more registers per thread (two CTAs) the kernel was measured at 5.7 / 5.2 TB/s (pack / unpack,
// frame sizes of 1 to 4 KB in 4 KB slots) with 21 % of the warp slots in use and its warps waiting on loads; capped at
// 64 registers it reaches 6.3 / 6.2 TB/s, the few spills sit in the unaligned fallback path.  (3 CTAs and 8 vectors in
// flight per lane: 6.4 / 5.9.)
#ifndef BLOAD_VAR_MIN_CTAS
#define BLOAD_VAR_MIN_CTAS 4
#endif
#ifndef BLOAD_VAR_UNROLL
#define BLOAD_VAR_UNROLL 4
#endif
template <bool UNPACK>
__global__ void __launch_bounds__(256, BLOAD_VAR_MIN_CTAS) k16_copy_var(PlanView pv, int32_t t_block, int32_t rows_max, int64_t row_stride,
                                                       int64_t block_begin, int64_t block_count,
                                                       const int32_t* __restrict__ seq_rows /*null: one row*/,
                                                       const int32_t* __restrict__ frame_bytes,
                                                       const int64_t* __restrict__ byte_offsets,
                                                       const uint8_t* __restrict__ src_base, uint8_t* __restrict__ dst_base,
                                                       int64_t sub_bytes, int64_t subs_per_block, uint8_t pad,
                                                       FastDiv div_vpr /*by row_stride / 16*/, FastDiv div_rows /*by rows_max*/)
{
    const int lane = threadIdx.x & 31;
    const bool rows_aligned = (row_stride & 15) == 0;  // every canvas row starts on a 16-byte boundary
    const uint32_t p4 = 0x01010101u * pad;
    const uint4 padv = make_uint4(p4, p4, p4, p4);
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_block;
    const int64_t slot_bytes = (int64_t)rows_max * row_stride;
    const int64_t block_bytes = (int64_t)t_block * slot_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int64_t ragged_total = byte_offsets[pv.hdr->n];
    const uint8_t* s_limit = src_base + (UNPACK ? block_count * block_bytes : ragged_total);

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
            if (cur < (int64_t)fill * slot_bytes) {
                // position inside the block: slot, canvas row, byte inside the row
                int slot = (int)(cur / slot_bytes);
                int r = (int)((cur - (int64_t)slot * slot_bytes) / row_stride);
                int64_t in = cur - (int64_t)slot * slot_bytes - (int64_t)r * row_stride;
                int k = warp_find_segment(pv.seg_start, k0, k1, slot, lane);
                int kw = k;  // lanes hold start slot, rows, row size and first byte of segments kw .. kw+31
                int w_st = fill, w_fb = 1, w_rows = 1;
                int64_t w_off = 0;
                auto load_window = [&]() {
                    w_st = fill; w_fb = 1; w_rows = 1; w_off = 0;
                    if (kw + lane < k1) {
                        const int id = pv.seg_seq[kw + lane];
                        w_st = pv.seg_start[kw + lane];
                        w_fb = (int)min((int64_t)max(frame_bytes[id], 1), row_stride);
                        w_rows = seq_rows ? min(max(seq_rows[id], 1), rows_max) : 1;
                        w_off = byte_offsets[id];
                    }
                };
                load_window();
                while (cur < hi && k < k1) {
                    if (k - kw == 31) { kw = k; load_window(); }
                    const int st = __shfl_sync(kFull, w_st, k - kw);
                    const int nx = __shfl_sync(kFull, w_st, k - kw + 1);
                    const int64_t fb = __shfl_sync(kFull, w_fb, k - kw);
                    const int rows = __shfl_sync(kFull, w_rows, k - kw);
                    const int64_t off = __shfl_sync(kFull, w_off, k - kw);
                    const int64_t seg_e = min((int64_t)nx * slot_bytes, hi);
                    if (fb == row_stride && rows == rows_max) {  // images fill their canvases: the segment is one run
                        const int64_t rag = off + (cur - (int64_t)st * slot_bytes);
                        if (UNPACK) warp_copy<true>(dst_base + rag, src_base + dense_off + cur, seg_e - cur, s_limit, lane);
                        else warp_copy<false>(dst_base + dense_off + cur, src_base + rag, seg_e - cur, s_limit, lane);
                        cur = seg_e;
                    } else if (rows_aligned && ((fb | off) & 15) == 0) {
                        // Rows of the store and of the canvases all start on 16-byte boundaries: one flat loop over the
                        // 16-byte vectors of [cur, seg_e) on the dense side.  A vector lies in canvas row `rr` of slot
                        // `sr` (both by the launch-constant divisions) and is either image data, which has its fixed
                        // place in the store, or padding; four independent vectors per lane are in flight.
                        const uint32_t nvec = (uint32_t)((seg_e - cur) >> 4);
                        const uint32_t c0 = (uint32_t)(in >> 4), fbv = (uint32_t)(fb >> 4), vpr = div_vpr.d;
                        const int64_t slot_rel0 = slot - st;
                        uint4* __restrict__ dv = reinterpret_cast<uint4*>((UNPACK ? const_cast<uint8_t*>(src_base) : dst_base) + dense_off + cur);
                        uint8_t* rag_seg = (UNPACK ? dst_base : const_cast<uint8_t*>(src_base)) + off;
                        auto locate = [&](uint32_t i, bool& data) -> uint4* {
                            const uint32_t ca = c0 + i;
                            const uint32_t jr = fast_div(ca, div_vpr);
                            const uint32_t c = ca - jr * vpr;
                            const uint32_t ra = (uint32_t)r + jr;
                            const uint32_t sr = fast_div(ra, div_rows);
                            const uint32_t rr = ra - sr * (uint32_t)rows_max;
                            data = rr < (uint32_t)rows && c < fbv;
                            return reinterpret_cast<uint4*>(rag_seg + ((slot_rel0 + sr) * rows + rr) * fb + 16 * (int64_t)c);
                        };
                        uint32_t i = lane;
                        constexpr int U = BLOAD_VAR_UNROLL;
                        for (; i + 32 * (U - 1) < nvec; i += 32 * U) {
                            uint4 v[U]; uint4* rp[U]; bool data[U];
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                rp[u] = locate(i + 32 * u, data[u]);
                                v[u] = padv;
                                if (data[u]) v[u] = ld_stream(UNPACK ? dv + i + 32 * u : rp[u]);
                            }
#pragma unroll
                            for (int u = 0; u < U; ++u) {
                                if (!UNPACK) st_stream(dv + i + 32 * u, v[u]);
                                else if (data[u]) st_stream(rp[u], v[u]);
                            }
                        }
                        for (; i < nvec; i += 32) {
                            bool data;
                            uint4* rp = locate(i, data);
                            if (!UNPACK) st_stream(dv + i, data ? ld_stream(rp) : padv);
                            else if (data) st_stream(rp, ld_stream(dv + i));
                        }
                        // where the walk stands after nvec vectors
                        const uint32_t ca = c0 + nvec, jr = fast_div(ca, div_vpr), ra = (uint32_t)r + jr, sr = fast_div(ra, div_rows);
                        in = (int64_t)(ca - jr * vpr) << 4;
                        r = (int)(ra - sr * (uint32_t)rows_max);
                        slot += (int)sr;
                        cur = seg_e;
                    } else {
                        while (cur < seg_e) {
                            if (r < rows && in < fb) {  // the image's part of this canvas row
                                const int64_t len = min(fb - in, seg_e - cur);
                                const int64_t rag = off + ((int64_t)(slot - st) * rows + r) * fb + in;
                                if (UNPACK) warp_copy<true>(dst_base + rag, src_base + dense_off + cur, len, s_limit, lane);
                                else warp_copy<false>(dst_base + dense_off + cur, src_base + rag, len, s_limit, lane);
                                cur += len; in += len;
                            }
                            if (cur < seg_e) {
                                // padding: the rest of this row, or, below the image, the rest of the canvas
                                const int64_t room = r < rows ? row_stride - in : (int64_t)(rows_max - r) * row_stride - in;
                                const int64_t len = min(room, seg_e - cur);
                                if (!UNPACK) warp_fill(dst_base + dense_off + cur, len, pad, lane);
                                cur += len; in += len;
                            }
                            if (in >= row_stride) {  // on to the next canvas row(s)
                                const int adv = (int)(in / row_stride);
                                in -= (int64_t)adv * row_stride;
                                r += adv;
                                if (r >= rows_max) { r = 0; ++slot; }
                            }
                        }
                    }
                    if (cur == (int64_t)nx * slot_bytes) { ++k; slot = nx; r = 0; in = 0; }
                }
            }
        }
        if (!UNPACK && cur < hi) warp_fill(dst_base + dense_off + cur, hi - cur, pad, lane);
    }
}

}  // namespace

cudaError_t launch_var_offsets(const int32_t* lengths, const int32_t* rows, const int32_t* frame_bytes, int64_t n,
                               int64_t* out, int64_t* max_rows, cudaStream_t st)
{
    count_launches(1);
    k15_var_offsets<<<1, kScanThreads, 0, st>>>(lengths, rows, frame_bytes, n, out, max_rows);
    return cudaPeekAtLastError();
}

cudaError_t launch_copy_var(bool unpack, const PlanView& pv, int32_t t_block, int32_t rows_max, int64_t row_stride,
                            int64_t block_begin, int64_t block_count, const int32_t* seq_rows, const int32_t* frame_bytes,
                            const int64_t* byte_offsets, const uint8_t* src, uint8_t* dst, uint8_t pad_byte, cudaStream_t st)
{
    if (block_count == 0) return cudaSuccess;
    const int64_t block_bytes = (int64_t)t_block * rows_max * row_stride;
    const int64_t sub = 16384;
    const int64_t spb = (block_bytes + sub - 1) / sub;
    const int64_t want = (block_count * spb + 7) / 8;
    const unsigned grid = (unsigned)(want < 0x7fffffffLL ? want : 0x7fffffffLL);
    // divisors of the kernel's flat vector loop (used when row_stride is a multiple of 16)
    auto make_div = [](uint32_t d) {
        FastDiv f;
        uint32_t l = 0;
        while ((1ull << l) < d) ++l;
        f.mul = (uint32_t)((((1ull << l) - d) << 32) / d + 1);
        f.sh1 = l < 1 ? l : 1;
        f.sh2 = l > 0 ? l - 1 : 0;
        f.d = d;
        return f;
    };
    const FastDiv div_vpr = make_div((uint32_t)(row_stride >= 16 && row_stride / 16 < 0x7fffffffLL ? row_stride / 16 : 1));
    const FastDiv div_rows = make_div((uint32_t)rows_max);
    count_launches(1);
#ifdef BLOAD_DEBUG
    {   // the size of the store is the last entry of the offsets on the device: the checking build may wait for it
        int64_t n = 0, total = 0;
        (void)cudaStreamSynchronize(st);
        (void)cudaMemcpy(&n, &pv.hdr->n, sizeof n, cudaMemcpyDeviceToHost);
        (void)cudaMemcpy(&total, byte_offsets + n, sizeof total, cudaMemcpyDeviceToHost);
        const size_t dense_bytes = (size_t)(block_count * block_bytes);
        if (unpack) BLOAD_DBG_EXPECT(st, dbg::kCopyVar, {{src, dense_bytes}}, {{dst, (size_t)total}});
        else BLOAD_DBG_EXPECT(st, dbg::kCopyVar, {{src, (size_t)total}}, {{dst, dense_bytes}});
    }
#endif
    note_copy_kernel(unpack ? kCallUnpackVar : kCallPackVar, unpack ? "k16_copy_var<unpack>" : "k16_copy_var<pack>");
    if (unpack)
        k16_copy_var<true><<<grid, 256, 0, st>>>(pv, t_block, rows_max, row_stride, block_begin, block_count, seq_rows,
                                                  frame_bytes, byte_offsets, src, dst, sub, spb, pad_byte, div_vpr, div_rows);
    else
        k16_copy_var<false><<<grid, 256, 0, st>>>(pv, t_block, rows_max, row_stride, block_begin, block_count, seq_rows,
                                                   frame_bytes, byte_offsets, src, dst, sub, spb, pad_byte, div_vpr, div_rows);
    return cudaPeekAtLastError();
}

}  // namespace bload

// Pack (ragged store -> dense blocks, with pad fill) and unpack (dense per-frame outputs -> ragged).
//
// Paper, Methods: the sequences assigned to a block are concatenated and the unfilled tail is padded
// with zeros.  Frames of one sequence are contiguous both in the ragged store and in its block, so
// the unit of copy is a run of T_i * frame_bytes bytes, not a frame: the kernels are a segmented
// memcpy driven by the plan's segment list and never touch per-slot metadata.
//
// Work decomposition: the dense side is cut into fixed-size byte ranges ("sub-tiles") so that work
// is balanced whatever the run lengths are (one run may span 100+ MB, another 32 bytes).  A warp
// owns a sub-tile: it locates the first overlapping segment with a 32-way cooperative search over
// the block's slice of the start table, keeps a 32-segment window of (start, source frame) in
// registers, and walks the runs.  Every run is moved with 16-byte loads and stores: the
// destination is brought to a 16-byte boundary with a few byte copies, and when source and
// destination are then misaligned relative to each other (frame sizes that are not multiples of
// 16, e.g. 4-byte tokens) each output vector is assembled from two aligned source vectors with
// funnel shifts.
#include "bload_internal.cuh"

namespace bload {

namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return __ldcs(p); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }

template <int U>
__device__ __forceinline__ void warp_copy_aligned(uint4* __restrict__ d, const uint4* __restrict__ s, int64_t nv, int lane)
{
    int64_t i = lane;
    for (; i + 32 * (U - 1) < nv; i += 32 * U) {
        uint4 r[U];
#pragma unroll
        for (int u = 0; u < U; ++u) r[u] = ld_stream(s + i + 32 * u);
#pragma unroll
        for (int u = 0; u < U; ++u) st_stream(d + i + 32 * u, r[u]);
    }
    for (; i < nv; i += 32) st_stream(d + i, ld_stream(s + i));
}

// Output vector j = bytes [16j + 4*WS + bits/8, +16) of the aligned source vectors a[j], a[j+1].
template <int WS>
__device__ __forceinline__ uint4 splice(uint4 a, uint4 b, int bits)
{
    const uint32_t w[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    uint4 o;
    o.x = __funnelshift_r(w[WS + 0], w[WS + 1], bits);
    o.y = __funnelshift_r(w[WS + 1], w[WS + 2], bits);
    o.z = __funnelshift_r(w[WS + 2], w[WS + 3], bits);
    o.w = __funnelshift_r(w[WS + 3], w[WS + 4], bits);
    return o;
}

template <int WS, int U>
__device__ __forceinline__ void warp_copy_shifted(uint4* __restrict__ d, const uint4* __restrict__ a, int64_t nv, int bits, int lane)
{
    int64_t i = lane;
    for (; i + 32 * (U - 1) < nv; i += 32 * U) {
        uint4 lo[U], hi[U];
#pragma unroll
        for (int u = 0; u < U; ++u) { lo[u] = ld_stream(a + i + 32 * u); hi[u] = ld_stream(a + i + 32 * u + 1); }
#pragma unroll
        for (int u = 0; u < U; ++u) st_stream(d + i + 32 * u, splice<WS>(lo[u], hi[u], bits));
    }
    for (; i < nv; i += 32) st_stream(d + i, splice<WS>(ld_stream(a + i), ld_stream(a + i + 1), bits));
}

// Copy n bytes; s_limit is the end of the whole source buffer (no load goes beyond it).
__device__ __forceinline__ void warp_copy(uint8_t* __restrict__ d, const uint8_t* __restrict__ s, int64_t n,
                                          const uint8_t* s_limit, int lane)
{
    int head = (int)((16u - (unsigned)(reinterpret_cast<uintptr_t>(d) & 15u)) & 15u);
    if ((int64_t)head > n) head = (int)n;
    if (lane < head) d[lane] = s[lane];
    d += head; s += head; n -= head;
    int64_t nv = n >> 4;
    const int sh = (int)(reinterpret_cast<uintptr_t>(s) & 15u);
    if (sh == 0) {
        warp_copy_aligned<4>(reinterpret_cast<uint4*>(d), reinterpret_cast<const uint4*>(s), nv, lane);
    } else {
        const uint8_t* a = s - sh;  // 16-byte aligned, not below the buffer start (the buffer is 16-byte aligned)
        const int64_t usable = ((s_limit - a) >> 4) - 1;  // vectors j with a[j+1] fully inside the buffer
        if (nv > usable) nv = usable > 0 ? usable : 0;
        const int bits = (sh & 3) * 8;
        uint4* dv = reinterpret_cast<uint4*>(d);
        const uint4* av = reinterpret_cast<const uint4*>(a);
        switch (sh >> 2) {
            case 0: warp_copy_shifted<0, 4>(dv, av, nv, bits, lane); break;
            case 1: warp_copy_shifted<1, 4>(dv, av, nv, bits, lane); break;
            case 2: warp_copy_shifted<2, 4>(dv, av, nv, bits, lane); break;
            default: warp_copy_shifted<3, 4>(dv, av, nv, bits, lane); break;
        }
    }
    for (int64_t t = (nv << 4) + lane; t < n; t += 32) d[t] = s[t];
}

__device__ __forceinline__ void warp_fill(uint8_t* __restrict__ d, int64_t n, uint8_t pad, int lane)
{
    int head = (int)((16u - (unsigned)(reinterpret_cast<uintptr_t>(d) & 15u)) & 15u);
    if ((int64_t)head > n) head = (int)n;
    if (lane < head) d[lane] = pad;
    d += head; n -= head;
    const int64_t nv = n >> 4;
    const uint32_t p4 = 0x01010101u * pad;
    const uint4 v = make_uint4(p4, p4, p4, p4);
    uint4* dv = reinterpret_cast<uint4*>(d);
    for (int64_t i = lane; i < nv; i += 32) st_stream(dv + i, v);
    for (int64_t t = (nv << 4) + lane; t < n; t += 32) d[t] = pad;
}

// Largest k in [k0, k1) with seg_start[k] <= slot (seg_start[k0] == 0 <= slot always holds).
__device__ __forceinline__ int warp_find_segment(const int32_t* __restrict__ seg_start, int k0, int k1, int slot, int lane)
{
    int lo = k0, hi = k1;
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) >> 5;
        const int idx = lo + lane * step;
        const bool p = idx < hi && seg_start[idx] <= slot;
        const int c = __popc(__ballot_sync(kFull, p));  // monotone: the first c lanes hold
        const int nlo = lo + (c - 1) * step;
        hi = min(hi, nlo + step);
        lo = nlo;
    }
    return lo;
}

template <bool UNPACK>
__global__ void __launch_bounds__(256) k7_copy(PlanView pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                                               int64_t block_count, const uint8_t* __restrict__ src_base,
                                               uint8_t* __restrict__ dst_base, int64_t src_total_bytes,
                                               int64_t sub_bytes, int64_t subs_per_block, uint8_t pad)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const uint8_t* s_limit = src_base + src_total_bytes;

    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_block;
        const int64_t lo = (item - q * subs_per_block) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, block_bytes);
        const int64_t b = block_begin + q;
        const int64_t dense_off = q * block_bytes;  // of this block inside the dense buffer
        int64_t cur = lo;
        if (b < n_blocks) {
            const int k0 = pv.block_seg_begin[b], k1 = pv.block_seg_begin[b + 1];
            const int fill = pv.block_fill[b];
            if (cur < (int64_t)fill * frame_bytes) {
                int k = warp_find_segment(pv.seg_start, k0, k1, (int)(cur / frame_bytes), lane);
                int kw = k;  // window base: lanes hold segments kw .. kw+31
                int w_st = (kw + lane < k1) ? pv.seg_start[kw + lane] : fill;
                int64_t w_src = (kw + lane < k1) ? pv.seg_src[kw + lane] : 0;
                while (cur < hi && k < k1) {
                    if (k - kw == 31) {
                        kw = k;
                        w_st = (kw + lane < k1) ? pv.seg_start[kw + lane] : fill;
                        w_src = (kw + lane < k1) ? pv.seg_src[kw + lane] : 0;
                    }
                    const int st = __shfl_sync(kFull, w_st, k - kw);
                    const int nx = __shfl_sync(kFull, w_st, k - kw + 1);
                    const int64_t src_frame = __shfl_sync(kFull, w_src, k - kw);
                    const int64_t seg_b = (int64_t)st * frame_bytes;
                    const int64_t pe = min((int64_t)nx * frame_bytes, hi);
                    const int64_t rag = src_frame * frame_bytes + (cur - seg_b);
                    if (UNPACK)
                        warp_copy(dst_base + rag, src_base + dense_off + cur, pe - cur, s_limit, lane);
                    else
                        warp_copy(dst_base + dense_off + cur, src_base + rag, pe - cur, s_limit, lane);
                    cur = pe;
                    ++k;
                }
            }
        }
        if (!UNPACK && cur < hi) warp_fill(dst_base + dense_off + cur, hi - cur, pad, lane);
    }
}

}  // namespace

cudaError_t launch_copy(bool unpack, const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                        int64_t block_count, const uint8_t* ragged_in, uint8_t* dense, uint8_t* ragged_out,
                        int64_t ragged_bytes, uint8_t pad_byte, cudaStream_t st)
{
    if (block_count == 0) return cudaSuccess;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t sub = 16384;
    const int64_t spb = (block_bytes + sub - 1) / sub;
    const int64_t items = block_count * spb;
    const int64_t want = (items + 7) / 8;
    const unsigned grid = (unsigned)(want < 148 * 8 ? want : 148 * 8);
    if (unpack)
        k7_copy<true><<<grid, 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count, dense, ragged_out,
                                             block_count * block_bytes, sub, spb, pad_byte);
    else
        k7_copy<false><<<grid, 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count, ragged_in, dense,
                                              ragged_bytes, sub, spb, pad_byte);
    count_launches(1);
    return cudaPeekAtLastError();
}

}  // namespace bload

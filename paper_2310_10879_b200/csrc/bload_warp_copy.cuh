// Warp-level building blocks of the copy kernels: a segmented memcpy in 16-byte vectors whatever the
// mutual alignment of source and destination, a pad fill, and the cooperative search of a block's
// slice of the start table.  Device code only; included by the translation units that move frames.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bload_debug.cuh"

namespace bload {
namespace wc {

constexpr unsigned kFull = 0xffffffffu;

// Every data access goes through these few functions; in a bounds-checking build (bload_debug.cuh) each asks first
// whether its address lies in a range the launcher registered, and a refused access is skipped.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) { return BLOAD_MAY_READ(p, 16) ? __ldcs(p) : make_uint4(0, 0, 0, 0); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { if (BLOAD_MAY_WRITE(p, 16)) __stcs(p, v); }
__device__ __forceinline__ void copy_byte(uint8_t* d, const uint8_t* s) { if (BLOAD_MAY_READ(s, 1) && BLOAD_MAY_WRITE(d, 1)) *d = *s; }
__device__ __forceinline__ void put_byte(uint8_t* d, uint8_t v) { if (BLOAD_MAY_WRITE(d, 1)) *d = v; }
__device__ __forceinline__ void put_word(uint8_t* d, uint32_t v) { if (BLOAD_MAY_WRITE(d, 4)) *reinterpret_cast<uint32_t*>(d) = v; }

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

// Loads of the realigning path: neighbouring lanes (and the two loads of one lane) touch the same 32-byte
// sectors.  Measured on B200 with 64..1028-byte frames: letting them allocate in L1 helps when the source is
// the dense side (unpack, +3..6 %) and costs when it is the ragged store (pack, -3..5 %), so the direction chooses.
template <bool CACHED>
__device__ __forceinline__ uint4 ld_shared_sector(const uint4* p)
{
    if (!BLOAD_MAY_READ(p, 16)) return make_uint4(0, 0, 0, 0);
    return CACHED ? __ldg(p) : __ldcs(p);
}

template <int WS, int U, bool CACHED>
__device__ __forceinline__ void warp_copy_shifted(uint4* __restrict__ d, const uint4* __restrict__ a, int64_t nv, int bits, int lane)
{
    int64_t i = lane;
    for (; i + 32 * (U - 1) < nv; i += 32 * U) {
        uint4 lo[U], hi[U];
#pragma unroll
        for (int u = 0; u < U; ++u) { lo[u] = ld_shared_sector<CACHED>(a + i + 32 * u); hi[u] = ld_shared_sector<CACHED>(a + i + 32 * u + 1); }
#pragma unroll
        for (int u = 0; u < U; ++u) st_stream(d + i + 32 * u, splice<WS>(lo[u], hi[u], bits));
    }
    for (; i < nv; i += 32) st_stream(d + i, splice<WS>(ld_shared_sector<CACHED>(a + i), ld_shared_sector<CACHED>(a + i + 1), bits));
}

// Copy n bytes; s_limit is the end of the whole source buffer (no load goes beyond it).
template <bool CACHED>
__device__ __forceinline__ void warp_copy(uint8_t* __restrict__ d, const uint8_t* __restrict__ s, int64_t n,
                                          const uint8_t* s_limit, int lane)
{
    int head = (int)((16u - (unsigned)(reinterpret_cast<uintptr_t>(d) & 15u)) & 15u);
    if ((int64_t)head > n) head = (int)n;
    if (lane < head) copy_byte(d + lane, s + lane);
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
            case 0: warp_copy_shifted<0, 4, CACHED>(dv, av, nv, bits, lane); break;
            case 1: warp_copy_shifted<1, 4, CACHED>(dv, av, nv, bits, lane); break;
            case 2: warp_copy_shifted<2, 4, CACHED>(dv, av, nv, bits, lane); break;
            default: warp_copy_shifted<3, 4, CACHED>(dv, av, nv, bits, lane); break;
        }
    }
    for (int64_t t = (nv << 4) + lane; t < n; t += 32) copy_byte(d + t, s + t);
}

__device__ __forceinline__ void warp_fill(uint8_t* __restrict__ d, int64_t n, uint8_t pad, int lane)
{
    int head = (int)((16u - (unsigned)(reinterpret_cast<uintptr_t>(d) & 15u)) & 15u);
    if ((int64_t)head > n) head = (int)n;
    if (lane < head) put_byte(d + lane, pad);
    d += head; n -= head;
    const int64_t nv = n >> 4;
    const uint32_t p4 = 0x01010101u * pad;
    const uint4 v = make_uint4(p4, p4, p4, p4);
    uint4* dv = reinterpret_cast<uint4*>(d);
    for (int64_t i = lane; i < nv; i += 32) st_stream(dv + i, v);
    for (int64_t t = (nv << 4) + lane; t < n; t += 32) put_byte(d + t, pad);
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

}  // namespace wc
}  // namespace bload

// Per-slot metadata of four consecutive slots of one block, shared by the metadata kernel and by the pack kernel that
// writes metadata from some of its CTAs.  Device code only.
#pragma once
#include "bload_debug.cuh"
#include "bload_internal.cuh"

namespace bload {

// Slots s0 .. s0+3 of block b (a filler block when b >= n_blocks); `o` is the index of slot s0 in the output arrays.
// VEC: t_block % 4 == 0 and aligned outputs, one vector store per array.
template <bool VEC>
__device__ __forceinline__ void metadata_quad(const PlanView& pv, int32_t t_block, int64_t b, int64_t n_blocks, int s0, int64_t o,
                                              int32_t* __restrict__ seq_id, int32_t* __restrict__ pos,
                                              uint8_t* __restrict__ reset, uint8_t* __restrict__ valid)
{
    const int32_t* __restrict__ seg_start = pv.seg_start;
    int sid[4] = {-1, -1, -1, -1}, ps[4] = {-1, -1, -1, -1};
    unsigned rs = 0, vd = 0;  // one flag byte per slot
    int fill = 0, k0 = 0, k1 = 0;
    if (b < n_blocks) {
        k0 = __ldg(pv.block_seg_begin + b);
        k1 = __ldg(pv.block_seg_begin + b + 1);
        fill = __ldg(pv.block_fill + b);
    }
    if (s0 < fill) {
        // last segment of the block that starts at or before s0 (seg_start[k0] == 0)
        int lo = k0, hi = k1;
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (__ldg(seg_start + mid) <= s0) lo = mid; else hi = mid;
        }
        int k = lo;
        int st = __ldg(seg_start + k);
        int nx = (k + 1 < k1) ? __ldg(seg_start + k + 1) : fill;
        int id = __ldg(pv.seg_seq + k);
        if (s0 + 3 < nx) {  // all four slots inside segment k
            const int p0 = s0 - st;
            sid[0] = sid[1] = sid[2] = sid[3] = id;
            ps[0] = p0; ps[1] = p0 + 1; ps[2] = p0 + 2; ps[3] = p0 + 3;
            vd = 0x01010101u;
            rs = p0 == 0 ? 1u : 0u;
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int s = s0 + e;
                if (s < fill) {
                    if (s >= nx) {
                        ++k;
                        st = nx;
                        nx = (k + 1 < k1) ? __ldg(seg_start + k + 1) : fill;
                        id = __ldg(pv.seg_seq + k);
                    }
                    sid[e] = id;
                    ps[e] = s - st;
                    vd |= 1u << (8 * e);
                    if (s == st) rs |= 1u << (8 * e);
                }
            }
        }
    }
    if (VEC) {  // t_block % 4 == 0 and aligned outputs: one vector per array
        if (seq_id && BLOAD_MAY_WRITE(seq_id + o, 16)) __stcs(reinterpret_cast<int4*>(seq_id + o), make_int4(sid[0], sid[1], sid[2], sid[3]));
        if (pos && BLOAD_MAY_WRITE(pos + o, 16)) __stcs(reinterpret_cast<int4*>(pos + o), make_int4(ps[0], ps[1], ps[2], ps[3]));
        if (reset && BLOAD_MAY_WRITE(reset + o, 4)) __stcs(reinterpret_cast<unsigned*>(reset + o), rs);
        if (valid && BLOAD_MAY_WRITE(valid + o, 4)) __stcs(reinterpret_cast<unsigned*>(valid + o), vd);
    } else {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (s0 + e < t_block) {
                if (seq_id && BLOAD_MAY_WRITE(seq_id + o + e, 4)) seq_id[o + e] = sid[e];
                if (pos && BLOAD_MAY_WRITE(pos + o + e, 4)) pos[o + e] = ps[e];
                if (reset && BLOAD_MAY_WRITE(reset + o + e, 1)) reset[o + e] = (uint8_t)((rs >> (8 * e)) & 1u);
                if (valid && BLOAD_MAY_WRITE(valid + o + e, 1)) valid[o + e] = (uint8_t)((vd >> (8 * e)) & 1u);
            }
        }
    }
}

}  // namespace bload

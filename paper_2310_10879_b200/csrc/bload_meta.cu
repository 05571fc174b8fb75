// Per-slot metadata: sequence id, position in sequence, reset flag at every sequence start,
// valid/pad mask (paper, Methods, second paragraph: the table of start indices, expanded per slot).
#include "bload_internal.cuh"

namespace bload {

namespace {

// One thread produces GROUP (4 or 16) consecutive slots of one block; groups never straddle blocks.
template <int GROUP, bool VEC>
__global__ void __launch_bounds__(256) k6_metadata(PlanView pv, int32_t t_block, int64_t block_begin,
                                                   int64_t block_count, int32_t groups_per_block,
                                                   int32_t* __restrict__ seq_id, int32_t* __restrict__ pos,
                                                   uint8_t* __restrict__ reset, uint8_t* __restrict__ valid)
{
    const int64_t total = block_count * (int64_t)groups_per_block;
    const int64_t n_blocks = pv.hdr->n_blocks;
    for (int64_t gidx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; gidx < total;
         gidx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t q = gidx / groups_per_block;
        const int s0 = (int)(gidx - q * groups_per_block) * GROUP;
        const int64_t b = block_begin + q;
        int sid[GROUP], ps[GROUP];
        unsigned rs[(GROUP + 3) / 4] = {0}, vd[(GROUP + 3) / 4] = {0};  // one flag byte per slot, packed 4 per word
#pragma unroll
        for (int e = 0; e < GROUP; ++e) { sid[e] = -1; ps[e] = -1; }
        if (b < n_blocks) {
            const int k0 = pv.block_seg_begin[b], k1 = pv.block_seg_begin[b + 1];
            const int fill = pv.block_fill[b];
            if (s0 < fill) {
                // last segment of the block that starts at or before s0
                int lo = k0, hi = k1;
                while (hi - lo > 1) {
                    int mid = (lo + hi) >> 1;
                    if (pv.seg_start[mid] <= s0) lo = mid; else hi = mid;
                }
                int k = lo;
                int st = pv.seg_start[k];
                int nx = (k + 1 < k1) ? pv.seg_start[k + 1] : fill;
                int id = pv.seg_seq[k];
#pragma unroll
                for (int e = 0; e < GROUP; ++e) {
                    const int s = s0 + e;
                    if (s < fill && s < t_block) {
                        if (s >= nx) {
                            ++k;
                            st = nx;
                            nx = (k + 1 < k1) ? pv.seg_start[k + 1] : fill;
                            id = pv.seg_seq[k];
                        }
                        sid[e] = id;
                        ps[e] = s - st;
                        vd[e >> 2] |= 1u << (8 * (e & 3));
                        if (s == st) rs[e >> 2] |= 1u << (8 * (e & 3));
                    }
                }
            }
        }
        const int64_t o = q * (int64_t)t_block + s0;
        if (VEC) {  // t_block % GROUP == 0, outputs aligned to GROUP elements
#pragma unroll
            for (int e = 0; e < GROUP; e += 4) {
                if (seq_id) *reinterpret_cast<int4*>(seq_id + o + e) = make_int4(sid[e], sid[e + 1], sid[e + 2], sid[e + 3]);
                if (pos) *reinterpret_cast<int4*>(pos + o + e) = make_int4(ps[e], ps[e + 1], ps[e + 2], ps[e + 3]);
            }
            if (GROUP == 16) {
                if (reset) *reinterpret_cast<uint4*>(reset + o) = make_uint4(rs[0], rs[1], rs[2], rs[3]);
                if (valid) *reinterpret_cast<uint4*>(valid + o) = make_uint4(vd[0], vd[1], vd[2], vd[3]);
            } else {
                if (reset) *reinterpret_cast<unsigned*>(reset + o) = rs[0];
                if (valid) *reinterpret_cast<unsigned*>(valid + o) = vd[0];
            }
        } else {
#pragma unroll
            for (int e = 0; e < GROUP; ++e) {
                if (s0 + e < t_block) {
                    if (seq_id) seq_id[o + e] = sid[e];
                    if (pos) pos[o + e] = ps[e];
                    if (reset) reset[o + e] = (uint8_t)((rs[e >> 2] >> (8 * (e & 3))) & 1u);
                    if (valid) valid[o + e] = (uint8_t)((vd[e >> 2] >> (8 * (e & 3))) & 1u);
                }
            }
        }
    }
}

}  // namespace

cudaError_t launch_metadata(const PlanView& pv, int32_t t_block, int64_t block_begin, int64_t block_count,
                            int32_t* seq_id, int32_t* pos, uint8_t* reset, uint8_t* valid, cudaStream_t st)
{
    if (block_count == 0) return cudaSuccess;
    auto al = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
    auto grid_for = [&](int group, int32_t* gpb) {
        *gpb = (t_block + group - 1) / group;
        const int64_t want = (block_count * (int64_t)*gpb + 255) / 256;
        return (unsigned)(want < 148 * 16 ? want : 148 * 16);
    };
    int32_t gpb;
    // (16 slots per thread with 16-byte flag stores was measured slower on B200: 2.30 ms against 1.83 ms for the
    // 8.75 GB of the token workload -- fewer threads, strided stores -- so 4 slots per thread it is)
    if (t_block % 4 == 0 && al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4)) {
        const unsigned grid = grid_for(4, &gpb);
        k6_metadata<4, true><<<grid, 256, 0, st>>>(pv, t_block, block_begin, block_count, gpb, seq_id, pos, reset, valid);
    } else {
        const unsigned grid = grid_for(4, &gpb);
        k6_metadata<4, false><<<grid, 256, 0, st>>>(pv, t_block, block_begin, block_count, gpb, seq_id, pos, reset, valid);
    }
    count_launches(1);
    return cudaPeekAtLastError();
}

}  // namespace bload

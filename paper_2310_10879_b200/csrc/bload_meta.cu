// Per-slot metadata: sequence id, position in sequence, reset flag at every sequence start,
// valid/pad mask (paper, Methods, second paragraph: the table of start indices, expanded per slot).
#include "bload_internal.cuh"

namespace bload {

namespace {

// One thread produces GROUP consecutive slots of one block; groups never straddle blocks.
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
        unsigned rs = 0, vd = 0;
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
                        vd |= 1u << (8 * e);
                        if (s == st) rs |= 1u << (8 * e);
                    }
                }
            }
        }
        const int64_t o = q * (int64_t)t_block + s0;
        if (VEC) {  // GROUP == 4, t_block % 4 == 0, outputs 16/4-byte aligned
            if (seq_id) *reinterpret_cast<int4*>(seq_id + o) = make_int4(sid[0], sid[1], sid[2], sid[3]);
            if (pos) *reinterpret_cast<int4*>(pos + o) = make_int4(ps[0], ps[1], ps[2], ps[3]);
            if (reset) *reinterpret_cast<unsigned*>(reset + o) = rs;
            if (valid) *reinterpret_cast<unsigned*>(valid + o) = vd;
        } else {
#pragma unroll
            for (int e = 0; e < GROUP; ++e) {
                if (s0 + e < t_block) {
                    if (seq_id) seq_id[o + e] = sid[e];
                    if (pos) pos[o + e] = ps[e];
                    if (reset) reset[o + e] = (uint8_t)((rs >> (8 * e)) & 1u);
                    if (valid) valid[o + e] = (uint8_t)((vd >> (8 * e)) & 1u);
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
    const int32_t gpb = (t_block + 3) / 4;
    const int64_t total = block_count * (int64_t)gpb;
    const int64_t want = (total + 255) / 256;
    const unsigned grid = (unsigned)(want < 148 * 16 ? want : 148 * 16);
    auto al = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
    const bool vec = (t_block % 4 == 0) && al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4);
    if (vec)
        k6_metadata<4, true><<<grid, 256, 0, st>>>(pv, t_block, block_begin, block_count, gpb, seq_id, pos, reset, valid);
    else
        k6_metadata<4, false><<<grid, 256, 0, st>>>(pv, t_block, block_begin, block_count, gpb, seq_id, pos, reset, valid);
    count_launches(1);
    return cudaPeekAtLastError();
}

}  // namespace bload

// Per-slot metadata: sequence id, position in sequence, reset flag at every sequence start,
// valid/pad mask (paper, Methods, second paragraph: the table of start indices, expanded per slot).
#include "bload_internal.cuh"

namespace bload {

namespace {

constexpr int kMetaThreads = 256;
constexpr int kMetaChunk = kMetaThreads * 4;  // slots of one block that a CTA produces per iteration

// A CTA produces chunks of kMetaChunk consecutive slots of one block: blockIdx.x is the chunk inside the block,
// blockIdx.y walks the blocks of the range (no per-thread division).  One thread produces 4 consecutive slots, so a
// warp writes 512 contiguous bytes of each id array and 128 of each flag array per store instruction.  The kernel
// writes 10 bytes per slot and is bound by instruction issue before it is bound by HBM, hence the fast path for
// the common case of four slots inside one segment.
template <bool VEC>
__global__ void __launch_bounds__(kMetaThreads) k6_metadata(PlanView pv, int32_t t_block, int64_t block_begin,
                                                            int32_t block_count, int32_t* __restrict__ seq_id,
                                                            int32_t* __restrict__ pos, uint8_t* __restrict__ reset,
                                                            uint8_t* __restrict__ valid, const int32_t* __restrict__ range)
{
    const int s0 = (int)blockIdx.x * kMetaChunk + (int)threadIdx.x * 4;
    if (s0 >= t_block) return;
    // `range` (device, or null): {first block, end block, end of the real blocks} of a plan that is still being built;
    // the outputs then start at block 0
    int64_t n_blocks, out_base = block_begin;
    if (range) { block_begin = range[0]; block_count = range[1] - range[0]; n_blocks = range[2]; out_base = 0; }
    else n_blocks = pv.hdr->n_blocks;
    const int32_t* __restrict__ seg_start = pv.seg_start;
    for (int q = blockIdx.y; q < block_count; q += gridDim.y) {
        const int64_t b = block_begin + q;
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
        const int64_t o = (b - out_base) * t_block + s0;
        if (VEC) {  // t_block % 4 == 0 and aligned outputs: one vector per array
            if (seq_id) __stcs(reinterpret_cast<int4*>(seq_id + o), make_int4(sid[0], sid[1], sid[2], sid[3]));
            if (pos) __stcs(reinterpret_cast<int4*>(pos + o), make_int4(ps[0], ps[1], ps[2], ps[3]));
            if (reset) __stcs(reinterpret_cast<unsigned*>(reset + o), rs);
            if (valid) __stcs(reinterpret_cast<unsigned*>(valid + o), vd);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
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
                            int32_t* seq_id, int32_t* pos, uint8_t* reset, uint8_t* valid, cudaStream_t st,
                            const int32_t* d_range)
{
    if (block_count == 0 && !d_range) return cudaSuccess;
    auto al = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
    const unsigned chunks = (unsigned)((t_block + kMetaChunk - 1) / kMetaChunk);
    // enough CTAs in flight to cover the machine several times over; beyond that a CTA loops over blocks
    int64_t rows = ((int64_t)device_info().sm_count * 64 + chunks - 1) / chunks;
    if (rows > block_count && !d_range) rows = block_count;
    if (d_range && rows > 256) rows = 256;  // a chunk of a plan in progress holds a few blocks
    if (rows > 65535) rows = 65535;
    const dim3 grid(chunks, (unsigned)rows);
    const size_t smem = d_range ? kBesideChainSmemBytes : 0;  // beside a running fill rule: stay off its SM
    if (t_block % 4 == 0 && al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4))
        k6_metadata<true><<<grid, kMetaThreads, smem, st>>>(pv, t_block, block_begin, (int32_t)block_count, seq_id, pos, reset, valid, d_range);
    else
        k6_metadata<false><<<grid, kMetaThreads, smem, st>>>(pv, t_block, block_begin, (int32_t)block_count, seq_id, pos, reset, valid, d_range);
    count_launches(1);
    return cudaPeekAtLastError();
}

}  // namespace bload

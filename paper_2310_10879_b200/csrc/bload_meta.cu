// Per-slot metadata: sequence id, position in sequence, reset flag at every sequence start,
// valid/pad mask (paper, Methods, second paragraph: the table of start indices, expanded per slot).
#include "bload_internal.cuh"
#include "bload_meta.cuh"

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
    for (int q = blockIdx.y; q < block_count; q += gridDim.y) {
        const int64_t b = block_begin + q;
        metadata_quad<VEC>(pv, t_block, b, n_blocks, s0, (b - out_base) * t_block + s0, seq_id, pos, reset, valid);
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
    if (d_range) {
        BLOAD_DBG_UNCHECKED(st);
    } else {
        [[maybe_unused]] const size_t slots = (size_t)block_count * (size_t)t_block;
        BLOAD_DBG_EXPECT(st, dbg::kMetadata, {}, {{seq_id, 4 * slots}, {pos, 4 * slots}, {reset, slots}, {valid, slots}});
    }
    if (t_block % 4 == 0 && al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4))
        k6_metadata<true><<<grid, kMetaThreads, smem, st>>>(pv, t_block, block_begin, (int32_t)block_count, seq_id, pos, reset, valid, d_range);
    else
        k6_metadata<false><<<grid, kMetaThreads, smem, st>>>(pv, t_block, block_begin, (int32_t)block_count, seq_id, pos, reset, valid, d_range);
    count_launches(1);
    return cudaPeekAtLastError();
}

}  // namespace bload

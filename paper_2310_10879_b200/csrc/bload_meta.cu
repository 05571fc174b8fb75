// Per-slot metadata: sequence id, position in sequence, reset flag at every sequence start,
// valid/pad mask (paper, Methods, second paragraph: the table of start indices, expanded per slot).
#include "bload_internal.cuh"
#include "bload_meta.cuh"
#include "bload_walk.cuh"

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
    release_dependents();
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

// The same outputs for blocks that are short or not a multiple of 4 slots long (the paper's own block of 94 frames): a
// thread produces 4 consecutive slots of the call's blocks taken as ONE array, wherever the blocks end, so every thread
// of a CTA has work (the kernel above gives a block a CTA of 1,024 slots at least: 9 % of it for 94 slots) and the ids
// leave in 16-byte vectors whatever t_block is.  A quad that runs into the next block carries on with its first segment.
template <bool VEC>
__global__ void __launch_bounds__(kMetaThreads) k6_metadata_flat(PlanView pv, int32_t t_block, int64_t block_begin, int64_t total,
                                                                 int32_t* __restrict__ seq_id, int32_t* __restrict__ pos,
                                                                 uint8_t* __restrict__ reset, uint8_t* __restrict__ valid)
{
    release_dependents();
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int32_t* __restrict__ seg_start = pv.seg_start;
    for (int64_t o = ((int64_t)blockIdx.x * kMetaThreads + threadIdx.x) * 4; o < total; o += (int64_t)gridDim.x * kMetaThreads * 4) {
        int64_t q = o / t_block;
        int s = (int)(o - q * t_block);
        int sid[4] = {-1, -1, -1, -1}, ps[4] = {-1, -1, -1, -1};
        unsigned rs = 0, vd = 0;  // one flag byte per slot
        int fill = 0, k = 0, k1 = 0, st = 0, nx = 0, id = 0;
        auto open_block = [&](int64_t b) {  // header of block b; its first segment starts at slot 0
            fill = 0; k = 0; k1 = 0;
            if (b < n_blocks) { k = __ldg(pv.block_seg_begin + b); k1 = __ldg(pv.block_seg_begin + b + 1); fill = __ldg(pv.block_fill + b); }
        };
        auto open_segment = [&]() {
            st = __ldg(seg_start + k);
            nx = (k + 1 < k1) ? __ldg(seg_start + k + 1) : fill;
            id = __ldg(pv.seg_seq + k);
        };
        open_block(block_begin + q);
        if (s < fill) {  // last segment of the block that starts at or before s
            int lo = k, hi = k1;
            while (hi - lo > 1) {
                const int mid = (lo + hi) >> 1;
                if (__ldg(seg_start + mid) <= s) lo = mid; else hi = mid;
            }
            k = lo;
            open_segment();
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (o + e < total) {
                if (s == t_block) {
                    ++q; s = 0;
                    open_block(block_begin + q);
                    if (fill > 0) open_segment();
                }
                if (s < fill) {
                    if (s >= nx) { ++k; open_segment(); }
                    sid[e] = id;
                    ps[e] = s - st;
                    vd |= 1u << (8 * e);
                    if (s == st) rs |= 1u << (8 * e);
                }
                ++s;
            }
        }
        if (VEC && o + 4 <= total) {
            if (seq_id && BLOAD_MAY_WRITE(seq_id + o, 16)) __stcs(reinterpret_cast<int4*>(seq_id + o), make_int4(sid[0], sid[1], sid[2], sid[3]));
            if (pos && BLOAD_MAY_WRITE(pos + o, 16)) __stcs(reinterpret_cast<int4*>(pos + o), make_int4(ps[0], ps[1], ps[2], ps[3]));
            if (reset && BLOAD_MAY_WRITE(reset + o, 4)) __stcs(reinterpret_cast<unsigned*>(reset + o), rs);
            if (valid && BLOAD_MAY_WRITE(valid + o, 4)) __stcs(reinterpret_cast<unsigned*>(valid + o), vd);
        } else {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (o + e < total) {
                    if (seq_id && BLOAD_MAY_WRITE(seq_id + o + e, 4)) seq_id[o + e] = sid[e];
                    if (pos && BLOAD_MAY_WRITE(pos + o + e, 4)) pos[o + e] = ps[e];
                    if (reset && BLOAD_MAY_WRITE(reset + o + e, 1)) reset[o + e] = (uint8_t)((rs >> (8 * e)) & 1u);
                    if (valid && BLOAD_MAY_WRITE(valid + o + e, 1)) valid[o + e] = (uint8_t)((vd >> (8 * e)) & 1u);
                }
            }
        }
    }
}

// Short runs (tens of slots): the two kernels above search the block's segment list once per quad, which costs more than
// the quad's 40 output bytes.  This one is the word-wise walk of the copy kernels (bload_walk.cuh) with a slot for a word:
// a warp takes 4,096 consecutive slots of the call's blocks as one array, lane l the quads l, l+32, ...; a lane finds the
// run of its quad in a window of 32 runs that the warp builds with one lane per run -- {begin of the next run, end,
// begin, sequence id} in slots relative to the warp's piece -- and only moves forward in it.  A quad inside one run (or
// inside padding) needs no search and no table load at all; a quad that holds the end of a run goes slot by slot.
constexpr int kMetaWalkSlots = 4096;  // slots per warp and turn, for calls that fill the machine
template <bool VEC>
__global__ void __launch_bounds__(256) k6_metadata_walk(PlanView pv, int32_t n, int32_t t_block, int64_t block_begin, int64_t total,
                                                        int32_t* __restrict__ seq_id, int32_t* __restrict__ pos,
                                                        uint8_t* __restrict__ reset, uint8_t* __restrict__ valid, int32_t piece)
{
    release_dependents();
    using namespace walk;
    __shared__ int4 windows[8][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int4* win = windows[warp];
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int64_t chunks = (total + piece - 1) / piece;
    for (int64_t c = (int64_t)blockIdx.x * 8 + warp; c < chunks; c += (int64_t)gridDim.x * 8) {
        const int64_t lo0 = c * (int64_t)piece;  // positions below are slots relative to this slot of the call
        const int p_end = (int)min((int64_t)piece, total - lo0);
        int kw = first_run_at(pv, n, block_begin, n_blocks, lo0, t_block, 1, lane);
        int r = 0, dn = 0, e = 0, b = 0, id = 0, d_last = 0, my_begin = 0;
        auto load_window = [&]() {  // one lane per run
            const int k = kw + lane;
            int4 w = make_int4(kFar, kFar, 0, -1);
            if (k < n) {
                const int blk = pv.seg_block[k], st = pv.seg_start[k];
                const int nst = k + 1 < n ? pv.seg_start[k + 1] : 0;  // a later run of the same block starts later
                const int e_slot = nst > st ? nst : pv.block_fill[blk];
                const int64_t d_flat = (blk - block_begin) * (int64_t)t_block + st - lo0;
                // (a run that began before this piece: in the same block, so more than -2^30; one before the call's blocks ends at
                // 0 and its begin is never used)
                const int64_t b_true = d_flat < -(1LL << 30) ? -(1LL << 30) : d_flat;
                w = make_int4(clamp_far(d_flat), clamp_far(d_flat + (e_slot - st)), b_true > (int64_t)kFar ? kFar : (int)b_true, pv.seg_seq[k]);
            }
            my_begin = w.x;
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; e = w0.y; b = w0.z; id = w0.w;
        };
        auto advance_to = [&](int s) {
            while (s >= dn) {  // (s < begin of the window's last entry, so r stays below 31)
                ++r;
                const int4 w = win[r];
                dn = w.x; e = w.y; b = w.z; id = w.w;
            }
        };
        load_window();
        int done = 0;  // a multiple of 4
        while (done < p_end) {
            // the quads of this turn: all whose slots lie before the begin of the window's last run (or before the end of the piece)
            const int limit = p_end <= d_last ? (p_end + 3) & ~3 : d_last & ~3;
            for (int q = done + 4 * lane; q < limit; q += 128) {
                int sid[4] = {-1, -1, -1, -1}, ps[4] = {-1, -1, -1, -1};
                unsigned rs = 0, vd = 0;  // one flag byte per slot
                advance_to(q);
                if (q + 4 <= e) {  // the quad lies inside the run
                    const int p0 = q - b;
                    sid[0] = sid[1] = sid[2] = sid[3] = id;
                    ps[0] = p0; ps[1] = p0 + 1; ps[2] = p0 + 2; ps[3] = p0 + 3;
                    vd = 0x01010101u;
                    rs = p0 == 0 ? 1u : 0u;
                } else if (!(q >= e && q + 4 <= dn)) {  // (else: inside padding, nothing to set)
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int sl = q + i;
                        if (sl < p_end) {
                            advance_to(sl);
                            if (sl < e) {
                                sid[i] = id;
                                ps[i] = sl - b;
                                vd |= 1u << (8 * i);
                                if (sl == b) rs |= 1u << (8 * i);
                            }
                        }
                    }
                }
                const int64_t o = lo0 + q;
                if (VEC && q + 4 <= p_end) {
                    if (seq_id && BLOAD_MAY_WRITE(seq_id + o, 16)) __stcs(reinterpret_cast<int4*>(seq_id + o), make_int4(sid[0], sid[1], sid[2], sid[3]));
                    if (pos && BLOAD_MAY_WRITE(pos + o, 16)) __stcs(reinterpret_cast<int4*>(pos + o), make_int4(ps[0], ps[1], ps[2], ps[3]));
                    if (reset && BLOAD_MAY_WRITE(reset + o, 4)) __stcs(reinterpret_cast<unsigned*>(reset + o), rs);
                    if (valid && BLOAD_MAY_WRITE(valid + o, 4)) __stcs(reinterpret_cast<unsigned*>(valid + o), vd);
                } else {
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        if (q + i < p_end) {
                            if (seq_id && BLOAD_MAY_WRITE(seq_id + o + i, 4)) seq_id[o + i] = sid[i];
                            if (pos && BLOAD_MAY_WRITE(pos + o + i, 4)) pos[o + i] = ps[i];
                            if (reset && BLOAD_MAY_WRITE(reset + o + i, 1)) reset[o + i] = (uint8_t)((rs >> (8 * i)) & 1u);
                            if (valid && BLOAD_MAY_WRITE(valid + o + i, 1)) valid[o + i] = (uint8_t)((vd >> (8 * i)) & 1u);
                        }
                    }
                }
            }
            done = limit;
            if (done < p_end) {
                // the next window opens with the run that holds slot `done` (or the last one before it): the last of this window's
                // runs that begins at or before it -- at least the 27th, since 31 runs of a slot or more lie before d_last
                kw += __popc(__ballot_sync(kFull, my_begin <= done)) - 1;
                load_window();
            }
        }
    }
}

}  // namespace

cudaError_t launch_metadata(const PlanView& pv, int32_t t_block, int64_t block_begin, int64_t block_count,
                            int32_t* seq_id, int32_t* pos, uint8_t* reset, uint8_t* valid, cudaStream_t st,
                            const int32_t* d_range, int64_t n, int64_t sum_t)
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
    // short runs: the walk (no search per quad).  Measured on B200, TB/s of the 10 bytes per slot, walk against the kernels
    // below: runs of 22 slots in blocks of 94: 4.19 against 3.65 (flat); runs of 58 slots in blocks of 10,000: 5.34 against
    // 4.51 (chunked); runs of 868 slots in blocks of 4,096: 6.56 against 6.75.
    constexpr int64_t kMetaWalkRun = 256;  // slots per run, on average, up to which the walk is used
    if (!d_range && n > 0 && n < 0x7fffff00LL && sum_t / n <= kMetaWalkRun) {
        const int64_t total = block_count * t_block;
        // (a piece of 4,096 slots per warp when that fills the machine, else a multiple of 512 slots, 512 at least)
        const int64_t per_warp = total / ((int64_t)device_info().sm_count * 32);
        const int piece = per_warp >= kMetaWalkSlots ? kMetaWalkSlots : (int)(per_warp < 512 ? 512 : ((per_warp + 511) / 512) * 512);
        const int64_t want = ((total + piece - 1) / piece + 7) / 8, cap = (int64_t)device_info().sm_count * 32;
        const unsigned walk_grid = (unsigned)(want < cap ? want : cap);
        if (al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4))
            k6_metadata_walk<true><<<walk_grid, 256, 0, st>>>(pv, (int32_t)n, t_block, block_begin, total, seq_id, pos, reset, valid, piece);
        else
            k6_metadata_walk<false><<<walk_grid, 256, 0, st>>>(pv, (int32_t)n, t_block, block_begin, total, seq_id, pos, reset, valid, piece);
        count_launches(1);
        return cudaPeekAtLastError();
    }
    // blocks that leave a CTA of the chunked kernel mostly idle, or whose length rules out its vector stores
    if (!d_range && (t_block % 4 != 0 || (int64_t)chunks * kMetaChunk * 4 > (int64_t)t_block * 5)) {
        const int64_t total = block_count * t_block;
        const int64_t want = (total + kMetaChunk - 1) / kMetaChunk, cap = (int64_t)device_info().sm_count * 64;
        const unsigned flat_grid = (unsigned)(want < cap ? want : cap);
        if (al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4))
            k6_metadata_flat<true><<<flat_grid, kMetaThreads, 0, st>>>(pv, t_block, block_begin, total, seq_id, pos, reset, valid);
        else
            k6_metadata_flat<false><<<flat_grid, kMetaThreads, 0, st>>>(pv, t_block, block_begin, total, seq_id, pos, reset, valid);
        count_launches(1);
        return cudaPeekAtLastError();
    }
    if (t_block % 4 == 0 && al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4))
        k6_metadata<true><<<grid, kMetaThreads, smem, st>>>(pv, t_block, block_begin, (int32_t)block_count, seq_id, pos, reset, valid, d_range);
    else
        k6_metadata<false><<<grid, kMetaThreads, smem, st>>>(pv, t_block, block_begin, (int32_t)block_count, seq_id, pos, reset, valid, d_range);
    count_launches(1);
    return cudaPeekAtLastError();
}

}  // namespace bload

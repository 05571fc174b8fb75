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
//
// In this file, in order:
//   k7_copy                      the register path described above (large frames, long runs)
//   k10 / k9 / k8                small word-sized frames, run by run through shared-memory stages (cp.async in, one bulk
//                                store out): pack, whole-plan unpack, unpack of a block sub-range
//   k17 / k18                    the same stages, word by word: runs of a few hundred bytes (a lane finds the run of each
//                                of its words in a window of 32 runs)
//   k19 / k21                    word by word without a stage: frames that are multiples of 8 bytes, and frames that are
//                                not multiples of 4 bytes in short runs
//   k24 / k25                    pack and whole-plan unpack of frames of 1 to 3 bytes in runs of 0.4 to 4 KB: the walk in
//                                granules of 16 bytes
//   k7b_copy_bulk                a measurement variant (large frames through the bulk-copy engine), off by default
//   launch_copy and friends      which kernel takes which call, with the measurements the rules come from
#include "bload_internal.cuh"
#include "bload_meta.cuh"
#include "bload_warp_copy.cuh"
#include "bload_walk.cuh"

namespace bload {

namespace {

using namespace wc;
using namespace walk;

// `range` (device, or null): {first block, end block, end of the real blocks} replaces block_begin / block_count /
// n_blocks when the blocks of a launch are decided on the device (a plan that is still being built); `out_base` is
// the block that the first row of the dense buffer holds.
template <bool UNPACK>
__global__ void __launch_bounds__(256) k7_copy(PlanView pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                                               int64_t block_count, const uint8_t* __restrict__ src_base,
                                               uint8_t* __restrict__ dst_base, int64_t src_total_bytes,
                                               int64_t sub_bytes, int64_t subs_per_block, uint8_t pad,
                                               const int32_t* __restrict__ range, int64_t out_base)
{
    const int lane = threadIdx.x & 31;
    const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    int64_t n_blocks;
    if (range) {
        block_begin = range[0]; block_count = range[1] - range[0]; n_blocks = range[2];
        if (!UNPACK) src_total_bytes = pv.hdr->sum_t * frame_bytes;  // the host does not know the size of the store yet
    } else {
        n_blocks = pv.hdr->n_blocks;
    }
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const uint8_t* s_limit = src_base + src_total_bytes;

    for (int64_t item = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); item < items; item += warps) {
        const int64_t q = item / subs_per_block;
        const int64_t lo = (item - q * subs_per_block) * sub_bytes;
        const int64_t hi = min(lo + sub_bytes, block_bytes);
        const int64_t b = block_begin + q;
        const int64_t dense_off = (b - out_base) * block_bytes;  // of this block inside the dense buffer
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
                        warp_copy<true>(dst_base + rag, src_base + dense_off + cur, pe - cur, s_limit, lane);
                    else
                        warp_copy<false>(dst_base + dense_off + cur, src_base + rag, pe - cur, s_limit, lane);
                    cur = pe;
                    ++k;
                }
            }
        }
        if (!UNPACK && cur < hi) warp_fill(dst_base + dense_off + cur, hi - cur, pad, lane);
    }
    if (!UNPACK) wait_for_prerequisites();  // (a pack launched beside the call's metadata kernel ends after it)
}


// ------------------------------------------------------------------------------------------------
// Staged kernels for small frames whose size is a multiple of 4 bytes (token ids, short feature
// vectors): runs are short and start at arbitrary 4-byte offsets, so the register path above keeps too
// few bytes in flight.  Here every warp owns a small ring of shared-memory stages, each the image of
// one aligned sub-tile:
//   k10_pack_contig    sub-tiles of the dense side: gather the runs into the stage with cp.async (16
//                      bytes where source and stage are mutually aligned, else 4 bytes), pad with
//                      shared-memory stores, write the sub-tile with one bulk copy (cp.async.bulk);
//   k9_unpack_ragged   whole-plan unpack, sub-tiles of the ragged side: same gather, from the blocks;
//   k8_unpack_staged   unpack of a block sub-range, sub-tiles of the dense side: load the valid part
//                      with 16-byte cp.async, scatter it to the ragged side with 16-byte stores.
// The loads of item i are in flight while item i-1 is completed, and nothing waits on a flag: the only
// waits are cp.async.wait_group / cp.async.bulk.wait_group, which end when the hardware copies end.
// Requires frame_bytes % 4 == 0 (and, for k8_unpack_staged, (t_block * frame_bytes) % 16 == 0).
// Tuning of the two directions (swept on B200 with the 4-byte token workload): bytes per stage, warps
// per CTA, stages per warp, consecutive sub-tiles of a block handled by one warp.  More, smaller stages
// mean more resident warps; the kernels are limited by per-warp instruction latency, not by bytes in flight.
#ifndef BLOAD_PACK_BYTES
#define BLOAD_PACK_BYTES 8192
#endif
#ifndef BLOAD_PACK_WARPS
#define BLOAD_PACK_WARPS 4
#endif
#ifndef BLOAD_PACK_STAGES
#define BLOAD_PACK_STAGES 2
#endif
#ifndef BLOAD_UNPACK_BYTES
#define BLOAD_UNPACK_BYTES 4096
#endif
#ifndef BLOAD_UNPACK_WARPS
#define BLOAD_UNPACK_WARPS 8
#endif
#ifndef BLOAD_UNPACK_STAGES
#define BLOAD_UNPACK_STAGES 2
#endif
#ifndef BLOAD_UNPACK_GROUP
#define BLOAD_UNPACK_GROUP 4
#endif
#pragma nv_diag_suppress 177  // (the pack configuration never reads kGroup)
template <int BYTES, int WARPS, int STAGES, int GROUP>
struct StageCfgT {
    static constexpr int kBytes = BYTES, kWarps = WARPS, kStages = STAGES, kGroup = GROUP;
    static_assert(BYTES % 512 == 0 && STAGES >= 2 && GROUP >= 1, "stage configuration");
};
#pragma nv_diag_default 177
struct StagedShape { int kBytes, kWarps, kStages; };  // a stage configuration as values, for the launch code
template <class C> constexpr StagedShape shape_of() { return StagedShape{C::kBytes, C::kWarps, C::kStages}; }
template <bool UNPACK> struct StageCfg : StageCfgT<BLOAD_PACK_BYTES, BLOAD_PACK_WARPS, BLOAD_PACK_STAGES, 2> {};
template <> struct StageCfg<true> : StageCfgT<BLOAD_UNPACK_BYTES, BLOAD_UNPACK_WARPS, BLOAD_UNPACK_STAGES, BLOAD_UNPACK_GROUP> {};
// the staged kernels win while the average run (T_i * frame_bytes) is short; measured cross-over on B200 at about
// 16 KB (1.4 KB runs: 6.0 against 3.8 TB/s; 14 KB: 5.9 against 5.8; 23 KB: 6.15 against 6.36)
#ifndef BLOAD_BULK_COPY
#define BLOAD_BULK_COPY 0
#endif
#ifndef BLOAD_STAGED_MAX_RUN
#define BLOAD_STAGED_MAX_RUN 16384
#endif
constexpr int64_t kStagedMaxRunBytes = BLOAD_STAGED_MAX_RUN;  // (-1: every frame size through the register path, to compare)
#ifndef BLOAD_PACK_CHUNK_TILES
#define BLOAD_PACK_CHUNK_TILES 4
#endif
constexpr int64_t kPackChunkTiles = BLOAD_PACK_CHUNK_TILES;  // consecutive sub-tiles a warp packs before it jumps ahead

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async4(uint32_t s, const void* g)
{
    if (!BLOAD_MAY_READ(g, 4)) return;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(s), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t s, const void* g)
{
    if (!BLOAD_MAY_READ(g, 8)) return;
    asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(s), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t s, const void* g)
{
    if (!BLOAD_MAY_READ(g, 16)) return;
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s), "l"(g) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void bulk_store(void* g, uint32_t s, uint32_t bytes)
{
    if (!BLOAD_MAY_WRITE(g, bytes)) return;
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(g), "r"(s), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory"); }

// four copies of `sz` bytes, 32 lanes apart, with immediate offsets
#define BLOAD_CP4X(op, sz, s, g, st)                                                                                \
    if (BLOAD_MAY_READ(g, sz) && BLOAD_MAY_READ((g) + 3 * st, sz))                                                  \
    asm volatile(op " [%0], [%1], " #sz ";\n\t" op " [%0+" #st "], [%1+" #st "], " #sz ";\n\t"                       \
                 op " [%0+2*" #st "], [%1+2*" #st "], " #sz ";\n\t" op " [%0+3*" #st "], [%1+3*" #st "], " #sz ";"   \
                 ::"r"(s), "l"(g) : "memory")

// asynchronous gather of n bytes (n % 4 == 0, both addresses 4-byte aligned) into shared memory
__device__ __forceinline__ void warp_gather_async(uint32_t sd, const uint8_t* __restrict__ gs, int n, int lane)
{
    if (((sd ^ (uint32_t)reinterpret_cast<uintptr_t>(gs)) & 15u) == 0) {
        int hw = (int)(((16u - (sd & 15u)) & 15u) >> 2);
        if (hw * 4 > n) hw = n >> 2;
        if (lane < hw) cp_async4(sd + 4 * lane, gs + 4 * lane);
        sd += 4 * hw; gs += 4 * hw; n -= 4 * hw;
        const int nv = n >> 4;
        {
            uint32_t s = sd + 16 * lane;
            const uint8_t* g = gs + 16 * lane;
            int rem = nv - lane;  // vectors left for this lane, 32 apart
            for (; rem > 96; rem -= 128, s += 2048, g += 2048) BLOAD_CP4X("cp.async.cg.shared.global", 16, s, g, 512);
            for (; rem > 0; rem -= 32, s += 512, g += 512) cp_async16(s, g);
        }
        const int tw = (n - (nv << 4)) >> 2;
        if (lane < tw) cp_async4(sd + (nv << 4) + 4 * lane, gs + (nv << 4) + 4 * lane);
    } else if (((sd ^ (uint32_t)reinterpret_cast<uintptr_t>(gs)) & 7u) == 0) {
        // source and stage agree modulo 8: one leading word to reach an 8-byte boundary, then 8-byte copies
        const int hw = (n >= 4) ? (int)((sd >> 2) & 1u) : 0;
        if (hw && lane == 0) cp_async4(sd, gs);
        if (hw) { sd += 4; gs += 4; n -= 4; }
        const int nd = n >> 3;
        uint32_t s = sd + 8 * lane;
        const uint8_t* g = gs + 8 * lane;
        int rem = nd - lane;  // double words left for this lane, 32 apart
        for (; rem > 96; rem -= 128, s += 1024, g += 1024) BLOAD_CP4X("cp.async.ca.shared.global", 8, s, g, 256);
        for (; rem > 0; rem -= 32, s += 256, g += 256) cp_async8(s, g);
        if ((n & 4) && lane == 0) cp_async4(sd + (nd << 3), gs + (nd << 3));
    } else {
        uint32_t s = sd + 4 * lane;
        const uint8_t* g = gs + 4 * lane;
        int rem = (n >> 2) - lane;  // words left for this lane, 32 apart
        for (; rem > 96; rem -= 128, s += 512, g += 512) BLOAD_CP4X("cp.async.ca.shared.global", 4, s, g, 128);
        for (; rem > 0; rem -= 32, s += 128, g += 128) cp_async4(s, g);
    }
}

template <int WS>
__device__ __forceinline__ void scatter_vectors(uint4* __restrict__ d, const uint4* __restrict__ a, int nv, int lane)
{
    int i = lane;
    for (; i + 96 < nv; i += 128) {  // four output vectors in flight per lane
        uint4 lo[4], hi[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { lo[u] = a[i + 32 * u]; if (WS) hi[u] = a[i + 32 * u + 1]; }
#pragma unroll
        for (int u = 0; u < 4; ++u) st_stream(d + i + 32 * u, WS ? splice<WS>(lo[u], hi[u], 0) : lo[u]);
    }
    for (; i < nv; i += 32) st_stream(d + i, WS ? splice<WS>(a[i], a[i + 1], 0) : a[i]);
}

// scatter of n bytes (n % 4 == 0, 4-byte aligned) from shared memory to global memory, with 16-byte
// stores on the global side; a misaligned shared-memory source is read as two aligned vectors per
// output vector (the second may reach up to 12 bytes past the run: the stage area has 16 spare bytes)
__device__ __forceinline__ void warp_scatter(uint8_t* __restrict__ gd, const uint8_t* __restrict__ ss, int n, int lane)
{
    int hw = (int)(((16u - (unsigned)(reinterpret_cast<uintptr_t>(gd) & 15u)) & 15u) >> 2);
    if (hw * 4 > n) hw = n >> 2;
    if (lane < hw) put_word(gd + 4 * lane, reinterpret_cast<const uint32_t*>(ss)[lane]);
    gd += 4 * hw; ss += 4 * hw; n -= 4 * hw;
    const int nv = n >> 4;
    uint4* d = reinterpret_cast<uint4*>(gd);
    const int ws = (int)((smem_addr(ss) & 15u) >> 2);  // word shift of the source, 0..3
    const uint4* a = reinterpret_cast<const uint4*>(ss - 4 * ws);
    switch (ws) {
        case 0: scatter_vectors<0>(d, a, nv, lane); break;
        case 1: scatter_vectors<1>(d, a, nv, lane); break;
        case 2: scatter_vectors<2>(d, a, nv, lane); break;
        default: scatter_vectors<3>(d, a, nv, lane); break;
    }
    const int tw = (n - (nv << 4)) >> 2;
    if (lane < tw) put_word(gd + (nv << 4) + 4 * lane, reinterpret_cast<const uint32_t*>(ss + (nv << 4))[lane]);
}

// What a warp has to remember about a sub-tile between its two phases.
struct StagedItem {
    int64_t dense_off;  // byte offset of [lo, hi) inside the dense buffer
    int lo;             // byte offset inside the block (blocks of the staged path are < 2^31 bytes)
    int nbytes;         // hi - lo
    int valid;          // bytes of [lo, hi) that hold frames (the rest is padding)
    bool fresh;         // first sub-tile of its group: the run walker restarts from the fields below
    int k, k1, fill;    // first overlapping segment, end of the block's segments, occupied slots
    int w_st;           // lane's entry of the 32-segment window starting at k: start slot ...
    int64_t w_src;      // ... and first source frame
};
struct GroupHeader { int k0, k1, fill; };
// Position of a warp in the segment list while it walks consecutive sub-tiles of one block.
struct RunWalker { int k, kw, k1, fill, w_st; int64_t w_src; };

__global__ void __launch_bounds__(StageCfg<true>::kWarps * 32) k8_unpack_staged(PlanView pv, int32_t t_block, int64_t frame_bytes,
                                                             int64_t block_begin, uint32_t groups,
                                                             const uint8_t* __restrict__ src_base,
                                                             uint8_t* __restrict__ dst_base, uint32_t groups_per_block,
                                                             uint8_t pad)
{
    // A group is kStageGroup consecutive sub-tiles of one block, handled by one warp so that the
    // position in the segment list carries over from one sub-tile to the next.
    // groups = blocks of this launch * groups_per_block < 2^31 (the launcher splits larger calls).
    using Cfg = StageCfg<true>;
    constexpr int NST = Cfg::kStages, kStageBytes = Cfg::kBytes, kStageWarps = Cfg::kWarps, kStageGroup = Cfg::kGroup;
    extern __shared__ __align__(128) uint8_t stage_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* my_stages = stage_mem + (size_t)warp * NST * kStageBytes;
    const uint32_t warps = gridDim.x * kStageWarps;
    const int fb = (int)frame_bytes;
    const int block_bytes = t_block * fb;
    const int64_t n_blocks = pv.hdr->n_blocks;

    // the three scalars of a group's block; loaded one group ahead so that their latency is hidden
    auto load_header = [&](uint32_t g) {
        GroupHeader h{0, 0, 0};
        const int64_t b = block_begin + g / groups_per_block;
        if (g < groups && b < n_blocks) {
            h.k0 = pv.block_seg_begin[b];
            h.k1 = pv.block_seg_begin[b + 1];
            h.fill = pv.block_fill[b];
        }
        return h;
    };
    RunWalker wk{0, 0, 0, 0, 0, 0};
    // walk the runs of a sub-tile; f(offset inside the sub-tile, byte offset in the ragged buffer, bytes)
    auto for_each_run = [&](const StagedItem& it, auto&& f) {
        if (it.fresh) { wk.k = wk.kw = it.k; wk.k1 = it.k1; wk.fill = it.fill; wk.w_st = it.w_st; wk.w_src = it.w_src; }
        const int hi = it.lo + it.valid;
        int cur = it.lo;
        while (cur < hi) {
            if (wk.k - wk.kw == 31) {
                wk.kw = wk.k;
                wk.w_st = (wk.kw + lane < wk.k1) ? pv.seg_start[wk.kw + lane] : wk.fill;
                wk.w_src = (wk.kw + lane < wk.k1) ? pv.seg_src[wk.kw + lane] : 0;
            }
            const int st = __shfl_sync(kFull, wk.w_st, wk.k - wk.kw);
            const int nx = __shfl_sync(kFull, wk.w_st, wk.k - wk.kw + 1);
            const int64_t src_frame = __shfl_sync(kFull, wk.w_src, wk.k - wk.kw);
            const int seg_e = nx * fb;
            const int pe = min(seg_e, hi);
            f(cur - it.lo, src_frame * fb + (cur - st * fb), pe - cur);
            cur = pe;
            if (pe == seg_e) ++wk.k;  // a run cut by the end of the sub-tile continues in the next one
        }
    };
    // second phase of an item whose loads have landed in `stage`
    auto complete = [&](const StagedItem& it, uint8_t* stage) {
        __syncwarp();
        for_each_run(it, [&](int off, int64_t rag, int n) { warp_scatter(dst_base + rag, stage + off, n, lane); });
        __syncwarp();  // all lanes are done reading before the stage is refilled
    };

    StagedItem prev;
    bool have_prev = false;
    int s = 0, s_prev = 0;
    uint32_t g = blockIdx.x * kStageWarps + warp;
    GroupHeader h_next = load_header(g);
    int wn_st = 0;          // prefetched window of the next group (when it starts at the top of a block)
    int64_t wn_src = 0;
    bool wn_valid = false;
    for (; g < groups; g += warps) {
        const GroupHeader h = h_next;
        h_next = load_header(g + warps);
        const uint32_t q = g / groups_per_block;
        const int first = (int)(g - q * groups_per_block) * kStageGroup;
        const int fill_bytes = h.fill * fb;
        int k = h.k0, w_st = wn_st;
        int64_t w_src = wn_src;
        if (!wn_valid) {
            const int lo0 = first * kStageBytes;
            if (lo0 != 0 && lo0 < fill_bytes) k = warp_find_segment(pv.seg_start, h.k0, h.k1, lo0 / fb, lane);
            w_st = (k + lane < h.k1) ? pv.seg_start[k + lane] : h.fill;
            w_src = (k + lane < h.k1) ? pv.seg_src[k + lane] : 0;
        }
        wn_valid = false;
#pragma unroll 1
        for (int j = 0; j < kStageGroup; ++j) {
            StagedItem it;
            it.lo = (first + j) * kStageBytes;
            if (it.lo >= block_bytes) break;
            it.nbytes = min(kStageBytes, block_bytes - it.lo);
            it.dense_off = (int64_t)q * block_bytes + it.lo;
            it.valid = it.lo < fill_bytes ? min(it.nbytes, fill_bytes - it.lo) : 0;
            it.fresh = j == 0;
            it.k = k; it.k1 = h.k1; it.fill = h.fill; it.w_st = w_st; it.w_src = w_src;
            if ((j == kStageGroup - 1 || it.lo + kStageBytes >= block_bytes) && g + warps < groups &&
                (g + warps) % groups_per_block == 0) {
                // the next group opens a block: its window does not need a search, fetch it now
                wn_st = (h_next.k0 + lane < h_next.k1) ? pv.seg_start[h_next.k0 + lane] : h_next.fill;
                wn_src = (h_next.k0 + lane < h_next.k1) ? pv.seg_src[h_next.k0 + lane] : 0;
                wn_valid = true;
            }
            uint8_t* stage = my_stages + (size_t)s * kStageBytes;
            const uint32_t sa = smem_addr(stage);
            {
                // whole vectors of the valid part: the sub-tile is 16-byte aligned and sized
                uint32_t sp = sa + 16 * lane;
                const uint8_t* gp = src_base + it.dense_off + 16 * lane;
                int rem = ((it.valid + 15) >> 4) - lane;
                for (; rem > 96; rem -= 128, sp += 2048, gp += 2048) BLOAD_CP4X("cp.async.cg.shared.global", 16, sp, gp, 512);
                for (; rem > 0; rem -= 32, sp += 512, gp += 512) cp_async16(sp, gp);
            }
            cp_async_commit();
            if (have_prev) {
                cp_async_wait<1>();  // everything but the group just committed has landed
                complete(prev, my_stages + (size_t)s_prev * kStageBytes);
            }
            prev = it; have_prev = true; s_prev = s;
            s = (s + 1 == NST) ? 0 : s + 1;
        }
    }
    if (have_prev) {
        cp_async_wait<0>();
        complete(prev, my_stages + (size_t)s_prev * kStageBytes);
    }
}


// ------------------------------------------------------------------------------------------------
// Whole-plan unpack for small word-sized frames, tiled on the RAGGED side.  When every block of the
// plan is unpacked, the ragged output is one contiguous buffer that is written completely, so it can
// be produced exactly like a pack: cut it into sub-tiles, gather each sub-tile's runs (now read from
// their blocks in the dense buffer, through the inverse tables seq_block / seq_start) into a
// shared-memory stage with cp.async, and write the stage with one bulk copy.  Every warp owns a
// contiguous range of sub-tiles: it locates its first sequence once (32-way search of `offsets`)
// and then only walks forward, 32 sequences per window.
__device__ __forceinline__ int warp_find_sequence(const int64_t* __restrict__ offsets, int n, int64_t frame, int lane)
{   // largest i in [0, n) with offsets[i] <= frame (offsets[0] == 0)
    int lo = 0, hi = n;
    while (hi - lo > 1) {
        const int step = (hi - lo + 31) >> 5;
        const int64_t idx = (int64_t)lo + (int64_t)lane * step;
        const bool p = idx < hi && offsets[idx] <= frame;
        const int c = __popc(__ballot_sync(kFull, p));
        const int nlo = lo + (c - 1) * step;
        hi = min(hi, nlo + step);
        lo = nlo;
    }
    return lo;
}

__global__ void __launch_bounds__(StageCfg<false>::kWarps * 32) k9_unpack_ragged(PlanView pv, int32_t n, int32_t t_block,
                                                                               int64_t frame_bytes, int64_t sum_t,
                                                                               const uint8_t* __restrict__ dense,
                                                                               uint8_t* __restrict__ ragged,
                                                                               int64_t tiles, int64_t tiles_per_warp)
{
    using Cfg = StageCfg<false>;
    constexpr int NST = Cfg::kStages, kStageBytes = Cfg::kBytes, kStageWarps = Cfg::kWarps;
    extern __shared__ __align__(128) uint8_t stage_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* my_stages = stage_mem + (size_t)warp * NST * kStageBytes;
    const int64_t gw = (int64_t)blockIdx.x * kStageWarps + warp;
    const int64_t t_begin = gw * tiles_per_warp;
    const int64_t t_end = min(t_begin + tiles_per_warp, tiles);
    if (t_begin >= t_end) return;
    const int64_t total = sum_t * frame_bytes;

    // window of 32 sequences from kw: first frame in the ragged order, first frame in the dense buffer
    int i = warp_find_sequence(pv.offsets, n, (t_begin * kStageBytes) / frame_bytes, lane);
    int kw = i;
    int64_t w_off = 0, w_src = 0;
    auto load_window = [&]() {
        const int s = kw + lane;
        w_off = s < n ? pv.offsets[s] : sum_t;  // the entry after the last sequence closes it
        w_src = s < n ? (int64_t)pv.seq_block[s] * t_block + pv.seq_start[s] : 0;
    };
    load_window();

    int64_t prev_lo = 0;
    int prev_n = 0, s = 0, s_prev = 0;
    bool have_prev = false;
    auto complete = [&](int64_t lo, int nbytes, uint8_t* stage) {
        fence_proxy_async();
        __syncwarp();
        const int n16 = nbytes & ~15;
        if (lane == 0 && n16) { bulk_store(ragged + lo, smem_addr(stage), (uint32_t)n16); bulk_commit(); }
        if (lane < nbytes - n16) put_byte(ragged + lo + n16 + lane, stage[n16 + lane]);  // last tile only: total % 16 bytes
    };
    for (int64_t t = t_begin; t < t_end; ++t) {
        uint8_t* stage = my_stages + (size_t)s * kStageBytes;
        const uint32_t sa = smem_addr(stage);
        const int64_t lo = t * kStageBytes;
        const int nbytes = (int)min((int64_t)kStageBytes, total - lo);
        if (lane == 0) bulk_wait_read<NST - 2>();  // the store that last read this stage has finished reading
        __syncwarp();
        int64_t cur = lo;
        const int64_t hi = lo + nbytes;
        while (cur < hi) {
            if (i - kw == 31) { kw = i; load_window(); }
            const int64_t off = __shfl_sync(kFull, w_off, i - kw);
            const int64_t nxt = __shfl_sync(kFull, w_off, i - kw + 1);
            const int64_t src = __shfl_sync(kFull, w_src, i - kw);
            const int64_t seq_e = nxt * frame_bytes;
            const int64_t pe = min(seq_e, hi);
            warp_gather_async(sa + (uint32_t)(cur - lo), dense + src * frame_bytes + (cur - off * frame_bytes), (int)(pe - cur), lane);
            cur = pe;
            if (pe == seq_e) ++i;
        }
        cp_async_commit();
        if (have_prev) {
            cp_async_wait<1>();
            complete(prev_lo, prev_n, my_stages + (size_t)s_prev * kStageBytes);
        }
        prev_lo = lo; prev_n = nbytes; have_prev = true; s_prev = s;
        s = (s + 1 == NST) ? 0 : s + 1;
    }
    cp_async_wait<0>();
    complete(prev_lo, prev_n, my_stages + (size_t)s_prev * kStageBytes);
    __syncwarp();
    if (lane == 0) bulk_wait_read<0>();
}

// ------------------------------------------------------------------------------------------------
// Pack for small word-sized frames with a contiguous range of dense sub-tiles per warp (the pack-side
// twin of k9_unpack_ragged).  The dense side of the call is cut into sub-tiles as ONE array, whatever the
// size of a block: a sub-tile may hold the end of one block, several whole small blocks and the start of
// another, and a block may begin at any 4-byte offset.  The warp locates its first segment once and then
// walks forward through the segment list, which runs on from one block to the next; only `fill` and the
// segment end of each new block are read, one block ahead.  Blocks at or beyond n_blocks are written as padding.
// META: the per-slot metadata of the same blocks comes out of the same launch.  The first `pack_ctas` CTAs pack; every
// further CTA writes the metadata of 4 x blockDim.x consecutive slots of one block (the code of the metadata kernel).
// A call for one training batch of small frames moves about a megabyte and is bound by launch overhead, so one launch
// instead of two is the gain; the two kinds of CTA run side by side on the machine.
struct MetaOut {
    int32_t* seq_id; int32_t* pos; uint8_t* reset; uint8_t* valid;
    uint32_t pack_ctas;        // CTAs of the grid that pack; the rest write metadata
    int32_t chunks_per_block;  // metadata CTAs per block
    int32_t vec;               // t_block % 4 == 0 and aligned outputs: vector stores
};
template <bool META>
__global__ void __launch_bounds__(StageCfg<false>::kWarps * 32) k10_pack_contig(PlanView pv, int32_t n, int32_t t_block,
                                                                              int64_t frame_bytes, int64_t block_begin,
                                                                              const uint8_t* __restrict__ store,
                                                                              uint8_t* __restrict__ dense, int64_t tiles,
                                                                              int64_t tiles_per_warp, int64_t total,
                                                                              uint8_t pad, MetaOut mo)
{
    using Cfg = StageCfg<false>;
    constexpr int NST = Cfg::kStages, kStageBytes = Cfg::kBytes, kStageWarps = Cfg::kWarps;
    if (META && blockIdx.x >= mo.pack_ctas) {
        const uint32_t m = blockIdx.x - mo.pack_ctas;
        const uint32_t q = m / (uint32_t)mo.chunks_per_block;
        const int s0 = (int)(m - q * (uint32_t)mo.chunks_per_block) * (kStageWarps * 32 * 4) + (int)threadIdx.x * 4;
        if (s0 < t_block) {
            const int64_t o = (int64_t)q * t_block + s0;
            if (mo.vec) metadata_quad<true>(pv, t_block, block_begin + q, pv.hdr->n_blocks, s0, o, mo.seq_id, mo.pos, mo.reset, mo.valid);
            else metadata_quad<false>(pv, t_block, block_begin + q, pv.hdr->n_blocks, s0, o, mo.seq_id, mo.pos, mo.reset, mo.valid);
        }
        return;
    }
    extern __shared__ __align__(128) uint8_t stage_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* my_stages = stage_mem + (size_t)warp * NST * kStageBytes;
    const int64_t gw = (int64_t)blockIdx.x * kStageWarps + warp;
    const int64_t n_warps = (int64_t)(META ? mo.pack_ctas : gridDim.x) * kStageWarps;
    const int fb = (int)frame_bytes;
    const int block_bytes = t_block * fb;
    const int64_t n_blocks = pv.hdr->n_blocks;
    auto seg_end_of = [&](int64_t b) { return b < n_blocks ? pv.block_seg_begin[b + 1] : 0; };
    auto fill_of = [&](int64_t b) { return b < n_blocks ? pv.block_fill[b] * fb : 0; };
    int64_t prev_off = 0;
    int prev_n = 0, s = 0, s_prev = 0;
    bool have_prev = false;
    // a finished sub-tile leaves with one bulk copy; only the very last sub-tile of a call can end off a 16-byte
    // boundary (total % 16 != 0), and its last words leave with plain stores
    auto complete = [&](int64_t off, int nbytes, uint8_t* stage) {
        fence_proxy_async();
        __syncwarp();
        const int nb16 = nbytes & ~15;
        if (lane == 0 && nb16) { bulk_store(dense + off, smem_addr(stage), (uint32_t)nb16); bulk_commit(); }
        if (lane < ((nbytes - nb16) >> 2)) put_word(dense + off + nb16 + 4 * lane, *reinterpret_cast<const uint32_t*>(stage + nb16 + 4 * lane));
    };
    const uint32_t p4 = 0x01010101u * pad;
    // padding bytes [p, pe) of a stage (both multiples of 4): words up to a 16-byte boundary, vectors, words
    auto fill_pad = [&](uint8_t* stage, int p, int pe) {
        const int a = min((p + 15) & ~15, pe);
        if (lane < ((a - p) >> 2)) *reinterpret_cast<uint32_t*>(stage + p + 4 * lane) = p4;
        const int bnd = max(a, pe & ~15);
        for (int o = a + 16 * lane; o < bnd; o += 512) *reinterpret_cast<uint4*>(stage + o) = make_uint4(p4, p4, p4, p4);
        if (lane < ((pe - bnd) >> 2)) *reinterpret_cast<uint32_t*>(stage + bnd + 4 * lane) = p4;
    };
    // the warp takes chunks of `tiles_per_warp` consecutive sub-tiles, chunk after chunk, grid-strided
    for (int64_t t_begin = gw * tiles_per_warp; t_begin < tiles; t_begin += n_warps * tiles_per_warp) {
    const int64_t t_end = min(t_begin + tiles_per_warp, tiles);
    const int64_t lo0 = t_begin * kStageBytes;
    int64_t q = lo0 / block_bytes;                   // block of this call the warp starts in
    int bo = (int)(q * block_bytes - lo0);           // where that block begins, relative to the sub-tile (<= 0 here)
    // current block: end of its segments and occupied bytes; the same two scalars of the next block
    int k1 = seg_end_of(block_begin + q), fill_bytes = fill_of(block_begin + q);
    int k1_next = seg_end_of(block_begin + q + 1), fill_next = fill_of(block_begin + q + 1);
    // position in the segment list and a window of 32 segments from kw (raw start slots, source frames)
    int k = (block_begin + q) < n_blocks ? pv.block_seg_begin[block_begin + q] : 0;
    if (bo != 0 && -bo < fill_bytes) k = warp_find_segment(pv.seg_start, k, k1, (-bo) / fb, lane);
    int kw = k, w_st = 0;
    int64_t w_src = 0;
    auto load_window = [&]() {
        const int si = kw + lane;
        w_st = si < n ? pv.seg_start[si] : 0;
        w_src = si < n ? pv.seg_src[si] : 0;
    };
    load_window();
    for (int64_t t = t_begin; t < t_end; ++t) {
        uint8_t* stage = my_stages + (size_t)s * kStageBytes;
        const uint32_t sa = smem_addr(stage);
        const int64_t lo = t * kStageBytes;
        const int nbytes = (int)min((int64_t)kStageBytes, total - lo);
        if (lane == 0) bulk_wait_read<NST - 2>();  // the store that last read this stage has finished reading
        __syncwarp();
        int p = 0;  // position in the sub-tile; the loop ends because every turn moves p or closes a block (block_bytes > 0)
        while (p < nbytes) {
            const int hi = min(bo + fill_bytes, nbytes);  // end of the block's frames, clipped
            while (p < hi) {
                if ((unsigned)(k - kw) >= 31u) { kw = k; load_window(); }
                const int st = __shfl_sync(kFull, w_st, k - kw);
                const int nx = __shfl_sync(kFull, w_st, k - kw + 1);
                const int64_t src = __shfl_sync(kFull, w_src, k - kw);
                const int seg_e = bo + ((k + 1 < k1) ? nx * fb : fill_bytes);  // the block's last run ends where its frames end
                const int pe = min(seg_e, hi);
                warp_gather_async(sa + (uint32_t)p, store + src * fb + (p - bo - st * fb), pe - p, lane);
                p = pe;
                if (pe == seg_e) ++k;
            }
            if (p < nbytes || bo + block_bytes == nbytes) {  // padding up to the end of the block, then the next block
                const int blk_end = bo + block_bytes;
                const int pe = min(blk_end, nbytes);
                fill_pad(stage, p, pe);
                p = pe;
                if (pe == blk_end) {  // the next block's segments follow directly in the list
                    ++q; bo = blk_end;
                    k = k1;  // (already there unless the warp started inside the padding of the block it leaves)
                    k1 = k1_next; fill_bytes = fill_next;
                    k1_next = seg_end_of(block_begin + q + 1); fill_next = fill_of(block_begin + q + 1);
                }
            }
        }
        bo -= nbytes;
        cp_async_commit();
        if (have_prev) {
            cp_async_wait<1>();
            complete(prev_off, prev_n, my_stages + (size_t)s_prev * kStageBytes);
        }
        prev_off = lo; prev_n = nbytes; have_prev = true; s_prev = s;
        s = (s + 1 == NST) ? 0 : s + 1;
    }
    }
    if (!have_prev) return;
    cp_async_wait<0>();
    complete(prev_off, prev_n, my_stages + (size_t)s_prev * kStageBytes);
    __syncwarp();
    if (lane == 0) bulk_wait_read<0>();
}


// ------------------------------------------------------------------------------------------------
// Runs of a few hundred bytes or less (short sentences of token ids, per-frame labels of short clips).  The kernels
// above hand one run at a time to the whole warp; with 40-word runs most lanes idle and the run's bookkeeping costs
// more than its copy.  Here the sub-tile is walked by WORDS instead: lane l takes the words l, l+32, ... of the
// stage-side array and finds the run of each of its words itself, in a window of 32 runs that the warp builds with one
// lane per run and keeps in shared memory.  A window entry holds where the run begins and ends in the stage-side
// array (relative to the first byte of the warp's range, clamped) and the distance from there to its source; a lane
// only ever moves forward in the window.  Every word costs the same dozen instructions whatever the run lengths are.
// Stages, completion and the sub-tile ranges per warp are those of k10_pack_contig / k9_unpack_ragged.
// stages of the word-wise kernels.  Swept on B200 (bytes x warps per CTA, two stages; pack / unpack TB/s): 4-byte frames in
// 232-byte runs 8 KB x 4: 2.64 / 3.29, 4 KB x 8: 3.54 / 3.56, 2 KB x 16: 3.32 / 3.49; 8-byte frames in 176-byte runs
// 2.81 / 3.28, 3.31 / 3.36, 3.84 / 3.28; 16-byte frames in 928-byte runs 5.65 / 5.36, 5.41 / 5.42, 5.46 / 5.24; 64-byte
// frames in 3.7 KB runs 5.97 / 5.85, 5.82 / 5.71, 5.92 / 5.65: narrow words want more warps, 16-byte words larger stages.
template <int W> struct ShortCfg : StageCfgT<4096, 8, 2, 2> {};
template <> struct ShortCfg<16> : StageCfgT<8192, 4, 2, 2> {};
constexpr int kShortWindowBytes = 32 * 16;
#ifndef BLOAD_SHORT_RUN
#define BLOAD_SHORT_RUN 768
#endif
#ifndef BLOAD_SHORT_CHUNK_TILES
#define BLOAD_SHORT_CHUNK_TILES 4
#endif
constexpr int64_t kShortChunkTiles = BLOAD_SHORT_CHUNK_TILES;  // consecutive sub-tiles a warp packs before it jumps ahead
// Short runs for the staged kernels: the word-wise ones (k17, k18) instead of the run-by-run ones (k10, k9).  Frames that
// are multiples of 8 bytes no longer reach these kernels through bload_pack / bload_unpack without metadata (the unstaged
// walks below are faster: see walks_unstaged); the single-launch pack with metadata still uses k17 for them, with 16-
// or 8-byte words.  Measured on B200 against k10_pack_contig / k9_unpack_ragged (pack / unpack, TB/s; word-wise first):
//   16-byte words: 16-byte frames in 352-byte runs 4.6 / 5.0 against 3.0 / 3.5, 32-byte frames in 704-byte runs 5.6 / 5.5
//     against 4.8 / 5.4, 64-byte frames in 3.7 KB runs 6.0 / 5.9 against 5.9 / 5.8, 16-byte frames in 14 KB runs 6.0 / 5.8
//     against 5.9 / 5.9;
//   4- and 8-byte words: 8-byte frames in 176-byte runs 3.3 / 3.4 against 1.5 / 1.9; 4-byte frames in 232-byte runs
//     3.6 / 3.6 against 2.4 / 2.3; 20-byte frames in 446-byte runs 4.4 / 4.4 against 3.3 / 4.0; 24-byte frames in 535-byte
//     runs 4.7 / 4.6 against 3.8 / 4.5; 12-byte frames in 696-byte runs 4.7 / 4.7 against 4.7 / 4.6; 40-byte frames in
//     892-byte runs 5.0 / 4.9 against 4.8 / 5.6; 20-byte frames in 1.2 KB runs 5.0 / 5.0 against 5.3 / 5.2; 4-byte frames
//     in 3.5 KB runs 5.0 / 5.2 against 5.8 / 6.0.
inline bool runs_are_short(int64_t ragged_bytes, int64_t n, int64_t frame_bytes)
{
    return frame_bytes % 16 == 0 || ragged_bytes / n <= BLOAD_SHORT_RUN;
}

// words [p0, p1) of the range, for the stage that images the range from t0; win[r] = {begin of run r+1, end, source minus
// stage-side position (64 bit)}; r, e, delta, dn are the lane's place in the window.  A word is W = 16, 8 or 4 bytes, the
// largest of them that divides the frame size: every run then begins and ends on a word boundary on both sides.
template <int W>
__device__ __forceinline__ void cp_async_word(uint32_t s, const void* g)
{
    if (W == 16) cp_async16(s, g);
    else if (W == 8) cp_async8(s, g);
    else cp_async4(s, g);
}
template <bool PAD, int W>
__device__ __forceinline__ void walk_words(const int4* __restrict__ win, int& r, int& e, int64_t& delta, int& dn, int p0, int p1,
                                           int t0, uint8_t* stage, const uint8_t* __restrict__ src, uint32_t p4, int lane)
{
    const uint32_t sa = smem_addr(stage);
    for (int p = p0 + W * lane; p < p1; p += 32 * W) {
        while (p >= dn) {  // (p < p1 <= begin of the window's last entry, so r stays below 31)
            ++r;
            const int4 w = win[r];  // {begin of the next run, end, source minus position}
            dn = w.x; e = w.y; delta = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
        }
        if (!PAD || p < e) cp_async_word<W>(sa + (uint32_t)(p - t0), src + delta + p);
        else if (W == 16) *reinterpret_cast<uint4*>(stage + (p - t0)) = make_uint4(p4, p4, p4, p4);
        else if (W == 8) *reinterpret_cast<uint2*>(stage + (p - t0)) = make_uint2(p4, p4);
        else *reinterpret_cast<uint32_t*>(stage + (p - t0)) = p4;
    }
}

template <bool META, int W>
__global__ void __launch_bounds__(ShortCfg<W>::kWarps * 32) k17_pack_short_runs(PlanView pv, int32_t n, int32_t t_block,
                                                                                  int64_t frame_bytes, int64_t block_begin,
                                                                                  const uint8_t* __restrict__ store,
                                                                                  uint8_t* __restrict__ dense, int64_t tiles,
                                                                                  int64_t tiles_per_warp, int64_t total,
                                                                                  uint8_t pad, MetaOut mo)
{
    using Cfg = ShortCfg<W>;
    constexpr int NST = Cfg::kStages, kStageBytes = Cfg::kBytes, kStageWarps = Cfg::kWarps;
    if (META && blockIdx.x >= mo.pack_ctas) {
        const uint32_t m = blockIdx.x - mo.pack_ctas;
        const uint32_t q = m / (uint32_t)mo.chunks_per_block;
        const int s0 = (int)(m - q * (uint32_t)mo.chunks_per_block) * (kStageWarps * 32 * 4) + (int)threadIdx.x * 4;
        if (s0 < t_block) {
            const int64_t o = (int64_t)q * t_block + s0;
            if (mo.vec) metadata_quad<true>(pv, t_block, block_begin + q, pv.hdr->n_blocks, s0, o, mo.seq_id, mo.pos, mo.reset, mo.valid);
            else metadata_quad<false>(pv, t_block, block_begin + q, pv.hdr->n_blocks, s0, o, mo.seq_id, mo.pos, mo.reset, mo.valid);
        }
        return;
    }
    extern __shared__ __align__(128) uint8_t stage_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* my_stages = stage_mem + (size_t)warp * NST * kStageBytes;
    int4* win = reinterpret_cast<int4*>(stage_mem + (size_t)kStageWarps * NST * kStageBytes + 16 + (size_t)warp * kShortWindowBytes);
    const int64_t gw = (int64_t)blockIdx.x * kStageWarps + warp;
    const int64_t n_warps = (int64_t)(META ? mo.pack_ctas : gridDim.x) * kStageWarps;
    const int fb = (int)frame_bytes;
    const int64_t block_bytes = (int64_t)t_block * fb;
    const int64_t n_blocks = pv.hdr->n_blocks;
    int64_t prev_off = 0;
    int prev_n = 0, s = 0, s_prev = 0;
    bool have_prev = false;
    auto complete = [&](int64_t off, int nbytes, uint8_t* stage) {
        fence_proxy_async();
        __syncwarp();
        const int nb16 = nbytes & ~15;
        if (lane == 0 && nb16) { bulk_store(dense + off, smem_addr(stage), (uint32_t)nb16); bulk_commit(); }
        if (lane < ((nbytes - nb16) >> 2)) put_word(dense + off + nb16 + 4 * lane, *reinterpret_cast<const uint32_t*>(stage + nb16 + 4 * lane));
    };
    const uint32_t p4 = 0x01010101u * pad;
    for (int64_t t_begin = gw * tiles_per_warp; t_begin < tiles; t_begin += n_warps * tiles_per_warp) {
        const int64_t t_end = min(t_begin + tiles_per_warp, tiles);
        const int64_t lo0 = t_begin * kStageBytes;  // positions below are relative to this byte of the call's dense side
        int kw = first_run_at(pv, n, block_begin, n_blocks, lo0, block_bytes, fb, lane);
        int r = 0, e = 0, dn = 0, d_last = 0;
        int64_t delta = 0;
        auto load_window = [&]() {  // one lane per run
            const int4 w = dense_side_entry(pv, n, kw + lane, block_begin, block_bytes, fb, lo0);
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; e = w0.y; delta = (int64_t)(((uint64_t)(uint32_t)w0.w << 32) | (uint32_t)w0.z);
        };
        load_window();
        for (int64_t t = t_begin; t < t_end; ++t) {
            uint8_t* stage = my_stages + (size_t)s * kStageBytes;
            const int64_t lo = t * kStageBytes;
            const int nbytes = (int)min((int64_t)kStageBytes, total - lo);
            const int t0 = (int)(lo - lo0), t1 = t0 + nbytes;
            if (lane == 0) bulk_wait_read<NST - 2>();  // the store that last read this stage has finished reading
            __syncwarp();
            int done = t0;
            while (done < t1) {  // ends: a turn reaches t1 or moves the window on by 31 runs that begin ever later
                const int limit = min(t1, d_last);
                walk_words<true, W>(win, r, e, delta, dn, done, limit, t0, stage, store, p4, lane);
                done = limit;
                if (limit == d_last) { kw += 31; load_window(); }
            }
            cp_async_commit();
            if (have_prev) {
                cp_async_wait<1>();
                complete(prev_off, prev_n, my_stages + (size_t)s_prev * kStageBytes);
            }
            prev_off = lo; prev_n = nbytes; have_prev = true; s_prev = s;
            s = (s + 1 == NST) ? 0 : s + 1;
        }
    }
    if (!have_prev) return;
    cp_async_wait<0>();
    complete(prev_off, prev_n, my_stages + (size_t)s_prev * kStageBytes);
    __syncwarp();
    if (lane == 0) bulk_wait_read<0>();
}

// whole-plan unpack, the ragged side walked by words (see k9_unpack_ragged for the tiling): a window entry is one
// sequence, which ends where the next begins
template <int W>
__global__ void __launch_bounds__(ShortCfg<W>::kWarps * 32) k18_unpack_short_runs(PlanView pv, int32_t n, int32_t t_block,
                                                                                    int64_t frame_bytes, int64_t sum_t,
                                                                                    const uint8_t* __restrict__ dense,
                                                                                    uint8_t* __restrict__ ragged,
                                                                                    int64_t tiles, int64_t tiles_per_warp)
{
    using Cfg = ShortCfg<W>;
    constexpr int NST = Cfg::kStages, kStageBytes = Cfg::kBytes, kStageWarps = Cfg::kWarps;
    extern __shared__ __align__(128) uint8_t stage_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* my_stages = stage_mem + (size_t)warp * NST * kStageBytes;
    int4* win = reinterpret_cast<int4*>(stage_mem + (size_t)kStageWarps * NST * kStageBytes + 16 + (size_t)warp * kShortWindowBytes);
    const int64_t gw = (int64_t)blockIdx.x * kStageWarps + warp;
    const int64_t t_begin = gw * tiles_per_warp;
    const int64_t t_end = min(t_begin + tiles_per_warp, tiles);
    if (t_begin >= t_end) return;
    const int64_t total = sum_t * frame_bytes;
    const int64_t lo0 = t_begin * kStageBytes;  // positions below are relative to this byte of the ragged side
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;

    int kw = warp_find_sequence(pv.offsets, n, lo0 / frame_bytes, lane);
    int r = 0, e = 0, dn = 0, d_last = 0;
    int64_t delta = 0;
    auto load_window = [&]() {
        const int i = kw + lane;
        int4 w = make_int4(kFar, kFar, 0, 0);
        if (i < n) {
            const int64_t d_flat = pv.offsets[i] * frame_bytes - lo0;
            const int64_t dl = pv.seq_block[i] * block_bytes + pv.seq_start[i] * frame_bytes - d_flat;
            w = make_int4(clamp_far(d_flat), kFar, (int)(uint32_t)(uint64_t)dl, (int)(uint32_t)((uint64_t)dl >> 32));
        }
        __syncwarp();  // every lane has left the previous window
        d_last = __shfl_sync(kFull, w.x, 31);
        win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
        __syncwarp();
        const int4 w0 = win[0];
        r = 0; dn = w0.x; e = w0.y; delta = (int64_t)(((uint64_t)(uint32_t)w0.w << 32) | (uint32_t)w0.z);
    };
    load_window();

    int64_t prev_lo = 0;
    int prev_n = 0, s = 0, s_prev = 0;
    bool have_prev = false;
    auto complete = [&](int64_t lo, int nbytes, uint8_t* stage) {
        fence_proxy_async();
        __syncwarp();
        const int n16 = nbytes & ~15;
        if (lane == 0 && n16) { bulk_store(ragged + lo, smem_addr(stage), (uint32_t)n16); bulk_commit(); }
        if (lane < ((nbytes - n16) >> 2)) put_word(ragged + lo + n16 + 4 * lane, *reinterpret_cast<const uint32_t*>(stage + n16 + 4 * lane));
    };
    for (int64_t t = t_begin; t < t_end; ++t) {
        uint8_t* stage = my_stages + (size_t)s * kStageBytes;
        const int64_t lo = t * kStageBytes;
        const int nbytes = (int)min((int64_t)kStageBytes, total - lo);
        const int t0 = (int)(lo - lo0), t1 = t0 + nbytes;
        if (lane == 0) bulk_wait_read<NST - 2>();  // the store that last read this stage has finished reading
        __syncwarp();
        int done = t0;
        while (done < t1) {
            const int limit = min(t1, d_last);
            walk_words<false, W>(win, r, e, delta, dn, done, limit, t0, stage, dense, 0u, lane);
            done = limit;
            if (limit == d_last) { kw += 31; load_window(); }
        }
        cp_async_commit();
        if (have_prev) {
            cp_async_wait<1>();
            complete(prev_lo, prev_n, my_stages + (size_t)s_prev * kStageBytes);
        }
        prev_lo = lo; prev_n = nbytes; have_prev = true; s_prev = s;
        s = (s + 1 == NST) ? 0 : s + 1;
    }
    cp_async_wait<0>();
    complete(prev_lo, prev_n, my_stages + (size_t)s_prev * kStageBytes);
    __syncwarp();
    if (lane == 0) bulk_wait_read<0>();
}

// The same walk along the dense side without a stage, in either direction.  Unpack (block sub-ranges with short runs):
// a lane loads each of its words from the dense side (lanes read consecutive words: coalesced) and stores it to the
// word's place in the ragged output (consecutive inside a run); words of padding are skipped.  Pack: the word comes from
// its place in the ragged store, or is padding, and goes to the dense side.  Words of 2 bytes and 1 byte serve frames
// that are not multiples of 4 bytes, which cp.async (4 bytes at least) cannot move.
template <int W, bool PACK>
__global__ void __launch_bounds__(256, 4) k19_walk_dense_side(PlanView pv, int32_t n, int32_t t_block, int64_t frame_bytes,
                                                           int64_t block_begin, const uint8_t* __restrict__ from,
                                                           uint8_t* __restrict__ to_base, int64_t total, uint8_t pad, int32_t piece)
{
    __shared__ int4 windows[8][32];
    constexpr int U = W == 16 ? 4 : 8;  // words in flight per lane (4-byte words, 232-byte runs: 2 -> 2.54, 4 -> 2.68, 8 -> 2.78 TB/s)
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int4* win = windows[warp];
    const int fb = (int)frame_bytes;
    const int64_t block_bytes = (int64_t)t_block * fb;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int64_t chunks = (total + piece - 1) / piece;
    const uint32_t p4 = 0x01010101u * pad;
    for (int64_t c = (int64_t)blockIdx.x * 8 + warp; c < chunks; c += (int64_t)gridDim.x * 8) {
        const int64_t lo0 = c * (int64_t)piece;  // positions below are relative to this byte of the call's dense side
        const int p_end = (int)min((int64_t)piece, total - lo0);
        int kw = first_run_at(pv, n, block_begin, n_blocks, lo0, block_bytes, fb, lane);
        int r = 0, e = 0, dn = 0, d_last = 0;
        int64_t delta = 0;
        auto load_window = [&]() {  // one lane per run
            const int4 w = dense_side_entry(pv, n, kw + lane, block_begin, block_bytes, fb, lo0);
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; e = w0.y; delta = (int64_t)(((uint64_t)(uint32_t)w0.w << 32) | (uint32_t)w0.z);
        };
        load_window();
        // the dense side of the chunk is read (unpack) or written (pack); the ragged side is the other one
        const uint8_t* dense_in = from + lo0;
        uint8_t* dense_out = to_base + lo0;
        int done = 0;
        while (done < p_end) {  // ends: a turn reaches p_end or moves the window on by 31 runs that begin ever later
            const int limit = min(p_end, d_last);
            for (int p = done + W * lane; p < limit; p += 32 * W * U) {
                int64_t at[U];   // the word's place on the ragged side
                bool ok[U];      // the word belongs to a run
                typename WordOf<W>::type v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = p + u * 32 * W;
                    ok[u] = false;
                    if (q < limit) {
                        while (q >= dn) {  // (q < limit <= begin of the window's last entry, so r stays below 31)
                            ++r;
                            const int4 w = win[r];  // {begin of the next run, end, source minus position}
                            dn = w.x; e = w.y; delta = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                        }
                        ok[u] = q < e;
                        at[u] = delta + q;
                    }
                }
                if (PACK) {
#pragma unroll
                    for (int u = 0; u < U; ++u) v[u] = ok[u] ? load_word<W>(from + at[u]) : pad_word<W>(p4);
#pragma unroll
                    for (int u = 0; u < U; ++u) if (p + u * 32 * W < limit) store_word<W>(dense_out + p + u * 32 * W, v[u]);
                } else {
#pragma unroll
                    for (int u = 0; u < U; ++u) if (ok[u]) v[u] = load_word<W>(dense_in + p + u * 32 * W);
#pragma unroll
                    for (int u = 0; u < U; ++u) if (ok[u]) store_word<W>(to_base + at[u], v[u]);
                }
            }
            done = limit;
            if (limit == d_last) { kw += 31; load_window(); }
        }
    }
}
// Pack of frames that are not multiples of 4 bytes in runs too long for the 2- and 1-byte words above: the same walk
// along the dense side in granules of 16 bytes.  A granule that lies inside one run -- nearly all of them, when runs
// last a kilobyte -- is two aligned 16-byte loads from wherever its source happens to begin, a byte shift and one
// 16-byte store; a granule of padding is one store; a granule that holds a run's end or begin is put together byte
// by byte from the window.  Against the register path the gain is in the short runs between the long ones: there a
// warp handles one run at a time and waits for its loads, here every lane has U granules of any runs in flight.
// A window is left at the last whole granule below its last entry and the next one starts at the run that holds that
// byte (a search, not a step of 31 runs); where 31 runs fill less than one granule, lanes 0..15 resolve that granule's
// bytes through the plan's tables directly.
__device__ __forceinline__ uint4 shift_bytes(uint4 a, uint4 b, int sh)  // bytes [sh, sh + 16) of a followed by b, 0 < sh < 16
{
    const int bits = (sh & 3) * 8;
    switch (sh >> 2) {
        case 0: return splice<0>(a, b, bits);
        case 1: return splice<1>(a, b, bits);
        case 2: return splice<2>(a, b, bits);
        default: return splice<3>(a, b, bits);
    }
}
// the byte at position `pos` of the call's dense side, from the tables alone (any lane, no window)
__device__ __forceinline__ uint8_t dense_byte(const PlanView& pv, int64_t block_begin, int64_t n_blocks, int64_t block_bytes, int fb,
                                              int64_t pos, const uint8_t* __restrict__ from, uint8_t pad)
{
    const int64_t q = pos / block_bytes, b = block_begin + q;
    if (b >= n_blocks) return pad;
    const int64_t in_block = pos - q * block_bytes;
    const int slot = (int)(in_block / fb);
    if (slot >= pv.block_fill[b]) return pad;
    int lo = pv.block_seg_begin[b], hi = pv.block_seg_begin[b + 1];  // the last run of the block that starts at or before slot
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pv.seg_start[mid] <= slot) lo = mid; else hi = mid;
    }
    const uint8_t* s = from + (pv.seg_src[lo] + (slot - pv.seg_start[lo])) * (int64_t)fb + (in_block - (int64_t)slot * fb);
    return BLOAD_MAY_READ(s, 1) ? *s : (uint8_t)0;
}
__global__ void __launch_bounds__(256, 4) k24_pack_granules(PlanView pv, int32_t n, int32_t t_block, int64_t frame_bytes,
                                                            int64_t block_begin, const uint8_t* __restrict__ from,
                                                            uint8_t* __restrict__ to_base, int64_t total, int64_t from_bytes,
                                                            uint8_t pad, int32_t piece)
{
    __shared__ int4 windows[8][32];
    constexpr int U = 4;  // granules in flight per lane
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int4* win = windows[warp];
    const int fb = (int)frame_bytes;
    const int64_t block_bytes = (int64_t)t_block * fb;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const int64_t chunks = (total + piece - 1) / piece;
    const uint32_t p4 = 0x01010101u * pad;
    const uint4 pad16 = make_uint4(p4, p4, p4, p4);
    const uint8_t* from_end = from + from_bytes;
    for (int64_t c = (int64_t)blockIdx.x * 8 + warp; c < chunks; c += (int64_t)gridDim.x * 8) {
        const int64_t lo0 = c * (int64_t)piece;  // positions below are relative to this byte of the call's dense side
        const int p_end = (int)min((int64_t)piece, total - lo0);
        uint8_t* dense_out = to_base + lo0;
        int r = 0, e = 0, dn = 0, d_last = 0;
        int64_t delta = 0;
        auto load_window = [&](int kw) {  // one lane per run
            const int4 w = dense_side_entry(pv, n, kw + lane, block_begin, block_bytes, fb, lo0);
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; e = w0.y; delta = (int64_t)(((uint64_t)(uint32_t)w0.w << 32) | (uint32_t)w0.z);
        };
        int done = 0;
        while (done < p_end) {
            load_window(first_run_at(pv, n, block_begin, n_blocks, lo0 + done, block_bytes, fb, lane));
            const int lim = min(p_end, d_last);
            const int lim_g = lim == p_end ? p_end : (lim & ~15);  // whole granules below the window's last entry
            if (lim_g <= done) {  // 31 runs inside one granule: its bytes one by one, from the tables
                const int cnt = min(16, p_end - done);
                if (lane < cnt) wc::put_byte(dense_out + done + lane, dense_byte(pv, block_begin, n_blocks, block_bytes, fb, lo0 + done + lane, from, pad));
                done += cnt;
                continue;
            }
            for (int p = done + 16 * lane; p < lim_g; p += 32 * 16 * U) {
                uint4 v0[U], v1[U];
                int kind[U];  // 0 nothing, 1 aligned source, 2 shifted source, 3 padding, 4 byte by byte
                int shv[U];   // kind 2: the source's offset in its 16-byte vector; kind 4: the window entry of the granule's first byte
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = p + u * 512;
                    kind[u] = 0; shv[u] = 0;
                    if (q < lim_g) {
                        while (q >= dn) {  // (q < lim_g <= begin of the window's last entry, so r stays below 31)
                            ++r;
                            const int4 w = win[r];
                            dn = w.x; e = w.y; delta = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                        }
                        const uint8_t* s = from + (delta + q);
                        const int sh = (int)(reinterpret_cast<uintptr_t>(s) & 15u);
                        if (q + 16 <= e && q + 16 <= p_end) {
                            if (sh == 0) { kind[u] = 1; v0[u] = wc::ld_stream(reinterpret_cast<const uint4*>(s)); }
                            else if (s - sh + 32 <= from_end) {
                                kind[u] = 2; shv[u] = sh;
                                v0[u] = wc::ld_shared_sector<false>(reinterpret_cast<const uint4*>(s - sh));
                                v1[u] = wc::ld_shared_sector<false>(reinterpret_cast<const uint4*>(s - sh) + 1);
                            } else { kind[u] = 4; shv[u] = r; }
                        } else if (q >= e && q + 16 <= dn && q + 16 <= p_end) kind[u] = 3;
                        else { kind[u] = 4; shv[u] = r; }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = p + u * 512;
                    uint4* d = reinterpret_cast<uint4*>(dense_out + q);
                    if (kind[u] == 1) wc::st_stream(d, v0[u]);
                    else if (kind[u] == 2) wc::st_stream(d, shift_bytes(v0[u], v1[u], shv[u]));
                    else if (kind[u] == 3) wc::st_stream(d, pad16);
                }
                // the granules that hold a run's begin or end: byte by byte, with a walk of their own from the granule's entry
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (kind[u] != 4) continue;
                    int rr = shv[u];
                    int4 w = win[rr];
                    int ddn = w.x, ee = w.y;
                    int64_t dd = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                    const int q = p + u * 512, q_end = min(q + 16, p_end);
                    for (int x = q; x < q_end; ++x) {
                        while (x >= ddn) {
                            ++rr; w = win[rr];
                            ddn = w.x; ee = w.y; dd = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                        }
                        if (x < ee) wc::copy_byte(dense_out + x, from + (dd + x));
                        else wc::put_byte(dense_out + x, pad);
                    }
                }
            }
            done = lim_g;
        }
    }
}
// Whole-plan unpack by the same unstaged walk, along the RAGGED side: a window entry is one sequence (it ends where the
// next begins), a lane loads each of its words from the word's place in the dense buffer and stores it in place; the
// stores are contiguous across the warp, the loads inside a run.
template <int W>
__global__ void __launch_bounds__(256, 4) k21_unpack_walk_ragged(PlanView pv, int32_t n, int32_t t_block, int64_t frame_bytes,
                                                              int64_t sum_t, const uint8_t* __restrict__ dense,
                                                              uint8_t* __restrict__ ragged, int32_t piece)
{
    __shared__ int4 windows[8][32];
    constexpr int U = W == 16 ? 4 : 8;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int4* win = windows[warp];
    const int64_t total = sum_t * frame_bytes;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t chunks = (total + piece - 1) / piece;
    for (int64_t c = (int64_t)blockIdx.x * 8 + warp; c < chunks; c += (int64_t)gridDim.x * 8) {
        const int64_t lo0 = c * (int64_t)piece;  // positions below are relative to this byte of the ragged side
        const int p_end = (int)min((int64_t)piece, total - lo0);
        int kw = warp_find_sequence(pv.offsets, n, lo0 / frame_bytes, lane);
        int r = 0, dn = 0, d_last = 0;
        int64_t delta = 0;
        auto load_window = [&]() {  // one lane per sequence
            const int i = kw + lane;
            int4 w = make_int4(kFar, kFar, 0, 0);
            if (i < n) {
                const int64_t d_flat = pv.offsets[i] * frame_bytes - lo0;
                const int64_t dl = pv.seq_block[i] * block_bytes + pv.seq_start[i] * frame_bytes - d_flat;
                w = make_int4(clamp_far(d_flat), kFar, (int)(uint32_t)(uint64_t)dl, (int)(uint32_t)((uint64_t)dl >> 32));
            }
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; delta = (int64_t)(((uint64_t)(uint32_t)w0.w << 32) | (uint32_t)w0.z);
        };
        load_window();
        uint8_t* out = ragged + lo0;
        int done = 0;
        while (done < p_end) {  // ends: a turn reaches p_end or moves the window on by 31 sequences that begin ever later
            const int limit = min(p_end, d_last);
            for (int p = done + W * lane; p < limit; p += 32 * W * U) {
                int64_t at[U];
                typename WordOf<W>::type v[U];
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = p + u * 32 * W;
                    if (q < limit) {
                        while (q >= dn) {  // (q < limit <= begin of the window's last entry, so r stays below 31)
                            ++r;
                            const int4 w = win[r];
                            dn = w.x; delta = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                        }
                        at[u] = delta + q;
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) if (p + u * 32 * W < limit) v[u] = load_word<W>(dense + at[u]);
#pragma unroll
                for (int u = 0; u < U; ++u) if (p + u * 32 * W < limit) store_word<W>(out + p + u * 32 * W, v[u]);
            }
            done = limit;
            if (limit == d_last) { kw += 31; load_window(); }
        }
    }
}
// Whole-plan unpack of the same frames in granules of 16 bytes, along the ragged side (which has no padding: every byte
// belongs to a sequence).  The stores are the aligned side here, the loads from the blocks the shifted one.
__device__ __forceinline__ uint8_t ragged_byte(const PlanView& pv, int n, int64_t block_bytes, int fb, int64_t pos,
                                               const uint8_t* __restrict__ dense)
{
    const int64_t f = pos / fb;
    int lo = 0, hi = n;  // the last sequence that begins at or before frame f
    while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (pv.offsets[mid] <= f) lo = mid; else hi = mid;
    }
    const uint8_t* s = dense + pv.seq_block[lo] * block_bytes + (pv.seq_start[lo] + (f - pv.offsets[lo])) * (int64_t)fb + (pos - f * fb);
    return BLOAD_MAY_READ(s, 1) ? *s : (uint8_t)0;
}
__global__ void __launch_bounds__(256, 4) k25_unpack_granules(PlanView pv, int32_t n, int32_t t_block, int64_t frame_bytes,
                                                              int64_t sum_t, const uint8_t* __restrict__ dense,
                                                              uint8_t* __restrict__ ragged, int64_t dense_bytes, int32_t piece)
{
    __shared__ int4 windows[8][32];
    constexpr int U = 4;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int4* win = windows[warp];
    const int fb = (int)frame_bytes;
    const int64_t total = sum_t * frame_bytes;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t chunks = (total + piece - 1) / piece;
    const uint8_t* dense_end = dense + dense_bytes;
    for (int64_t c = (int64_t)blockIdx.x * 8 + warp; c < chunks; c += (int64_t)gridDim.x * 8) {
        const int64_t lo0 = c * (int64_t)piece;  // positions below are relative to this byte of the ragged side
        const int p_end = (int)min((int64_t)piece, total - lo0);
        uint8_t* out = ragged + lo0;
        int r = 0, dn = 0, d_last = 0;
        int64_t delta = 0;
        auto load_window = [&](int kw) {  // one lane per sequence
            const int i = kw + lane;
            int4 w = make_int4(kFar, kFar, 0, 0);
            if (i < n) {
                const int64_t d_flat = pv.offsets[i] * frame_bytes - lo0;
                const int64_t dl = pv.seq_block[i] * block_bytes + pv.seq_start[i] * frame_bytes - d_flat;
                w = make_int4(clamp_far(d_flat), kFar, (int)(uint32_t)(uint64_t)dl, (int)(uint32_t)((uint64_t)dl >> 32));
            }
            __syncwarp();  // every lane has left the previous window
            d_last = __shfl_sync(kFull, w.x, 31);
            win[lane] = make_int4(__shfl_down_sync(kFull, w.x, 1), w.y, w.z, w.w);  // (lane 31's entry is never walked)
            __syncwarp();
            const int4 w0 = win[0];
            r = 0; dn = w0.x; delta = (int64_t)(((uint64_t)(uint32_t)w0.w << 32) | (uint32_t)w0.z);
        };
        int done = 0;
        while (done < p_end) {
            load_window(warp_find_sequence(pv.offsets, n, (lo0 + done) / frame_bytes, lane));
            const int lim = min(p_end, d_last);
            const int lim_g = lim == p_end ? p_end : (lim & ~15);  // whole granules below the window's last entry
            if (lim_g <= done) {  // 31 sequences inside one granule: its bytes one by one, from the tables
                const int cnt = min(16, p_end - done);
                if (lane < cnt) wc::put_byte(out + done + lane, ragged_byte(pv, n, block_bytes, fb, lo0 + done + lane, dense));
                done += cnt;
                continue;
            }
            for (int p = done + 16 * lane; p < lim_g; p += 32 * 16 * U) {
                uint4 v0[U], v1[U];
                int kind[U];  // 0 nothing, 1 aligned source, 2 shifted source, 4 byte by byte
                int shv[U];   // kind 2: the source's offset in its 16-byte vector; kind 4: the window entry of the granule's first byte
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const int q = p + u * 512;
                    kind[u] = 0; shv[u] = 0;
                    if (q < lim_g) {
                        while (q >= dn) {  // (q < lim_g <= begin of the window's last entry, so r stays below 31)
                            ++r;
                            const int4 w = win[r];
                            dn = w.x; delta = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                        }
                        const uint8_t* s = dense + (delta + q);
                        const int sh = (int)(reinterpret_cast<uintptr_t>(s) & 15u);
                        if (q + 16 <= dn && q + 16 <= p_end) {
                            if (sh == 0) { kind[u] = 1; v0[u] = wc::ld_stream(reinterpret_cast<const uint4*>(s)); }
                            else if (s - sh + 32 <= dense_end) {
                                kind[u] = 2; shv[u] = sh;
                                v0[u] = wc::ld_shared_sector<true>(reinterpret_cast<const uint4*>(s - sh));
                                v1[u] = wc::ld_shared_sector<true>(reinterpret_cast<const uint4*>(s - sh) + 1);
                            } else { kind[u] = 4; shv[u] = r; }
                        } else { kind[u] = 4; shv[u] = r; }
                    }
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    uint4* d = reinterpret_cast<uint4*>(out + p + u * 512);
                    if (kind[u] == 1) wc::st_stream(d, v0[u]);
                    else if (kind[u] == 2) wc::st_stream(d, shift_bytes(v0[u], v1[u], shv[u]));
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    if (kind[u] != 4) continue;
                    int rr = shv[u];
                    int4 w = win[rr];
                    int ddn = w.x;
                    int64_t dd = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                    const int q = p + u * 512, q_end = min(q + 16, p_end);
                    for (int x = q; x < q_end; ++x) {
                        while (x >= ddn) {
                            ++rr; w = win[rr];
                            ddn = w.x; dd = (int64_t)(((uint64_t)(uint32_t)w.w << 32) | (uint32_t)w.z);
                        }
                        wc::copy_byte(out + x, dense + (dd + x));
                    }
                }
            }
            done = lim_g;
        }
    }
}
using WalkRaggedKernel = void (*)(PlanView, int32_t, int32_t, int64_t, int64_t, const uint8_t*, uint8_t*, int32_t);
inline WalkRaggedKernel walk_ragged_kernel_for(int64_t frame_bytes)
{
    return frame_bytes % 16 == 0 ? k21_unpack_walk_ragged<16> : frame_bytes % 8 == 0 ? k21_unpack_walk_ragged<8>
           : frame_bytes % 4 == 0 ? k21_unpack_walk_ragged<4> : frame_bytes % 2 == 0 ? k21_unpack_walk_ragged<2>
                                                                                     : k21_unpack_walk_ragged<1>;
}

using WalkKernel = void (*)(PlanView, int32_t, int32_t, int64_t, int64_t, const uint8_t*, uint8_t*, int64_t, uint8_t, int32_t);
template <bool PACK>
WalkKernel walk_kernel_for(int64_t frame_bytes)
{
    return frame_bytes % 16 == 0 ? k19_walk_dense_side<16, PACK> : frame_bytes % 8 == 0 ? k19_walk_dense_side<8, PACK>
           : frame_bytes % 4 == 0 ? k19_walk_dense_side<4, PACK> : frame_bytes % 2 == 0 ? k19_walk_dense_side<2, PACK>
                                                                                        : k19_walk_dense_side<1, PACK>;
}
// Which calls take the unstaged walks (k19 along the dense side: pack and block sub-ranges; k21 along the ragged side:
// whole-plan unpack).  Measured on B200 over three length distributions, about 1.5 GB per case (TB/s, pack / whole-plan
// unpack, walk against the best of the staged kernels or the register path):
//   16-byte words: 16-byte frames in 352-byte runs 5.04 / 4.91 against 4.59 / 4.96; 32-byte frames in 1.9 KB runs
//     6.03 / 6.08 against 5.86 / 5.56; 256-byte frames in 15 KB runs 6.28 / 6.45 against 5.96 / 6.24; 16-byte frames in 14 KB
//     runs 6.22 / 6.37 against 5.88 / 6.06
//   8-byte words: 8-byte frames in 176-byte runs 3.92 / 3.83 against 3.36 / 3.40, in 464-byte runs 5.07 / 5.00 against
//     4.45 / 4.42, in 6.9 KB runs 6.22 / 6.20 against 5.83 / 5.75; 24-byte frames in 1.4 KB runs 5.90 / 5.80 against 5.58 / 5.37
//   4-byte words: 4-byte frames in 232-byte runs 3.61 / 3.66 against 3.59 / 3.65 (word-wise staged), 20-byte frames in
//     1.2 KB runs 4.93 / 4.98 against 5.25 / 5.25 (run by run), 4-byte frames in 3.5 KB runs 5.19 / 5.30 against 5.87 / 6.08:
//     the staged kernels keep the frames that are multiples of 4 but not of 8 bytes
//   2-byte words (frames that are even but not multiples of 4; against the register path): 6-byte frames in 133-byte runs
//     2.24 / 2.23 against 0.46 / 0.71, in 346-byte runs 2.85 / 2.95 against 1.26 / 1.88; 30-byte frames in 669-byte runs
//     3.16 / 3.24 against 1.68 / 2.34, in 1.7 KB runs 3.34 / 3.52 against 3.06 / 3.79; 2-byte frames in 1.7 KB runs 3.36 / 3.55
//     against 3.66 / 4.20
//   1-byte words (odd frame sizes): 3-byte frames in 173-byte runs 1.49 / 1.56 against 0.73 / 1.15; 1-byte frames in
//     870-byte runs 1.87 / 2.07 against 2.51 / 3.23
// Tried for the 4-byte words and dropped: the ragged-side walk in 16-byte groups (four 4-byte loads and one 16-byte store
// per group that lies inside one run, word by word for the groups that hold a run's end).  Whole-plan unpack, TB/s,
// against the staged kernels: 4-byte frames in 3.5 KB runs 5.86 against 6.10, 12-byte frames in 10 KB runs 6.07 against
// 6.06, 100-byte frames in 5.8 KB runs 5.99 against 6.04, 4-byte frames in 232-byte runs 3.75 against 3.65, 12-byte frames
// in 696-byte runs 4.97 against 4.70: within 6 % either way, so the staged kernels stayed.
#ifndef BLOAD_GRANULE_MAX_RUN
#define BLOAD_GRANULE_MAX_RUN 4096
#endif
#ifndef BLOAD_ODD_WALKS
#define BLOAD_ODD_WALKS 1  // 0: no 2- and 1-byte word walks (to compare the granule kernels with them)
#endif
#ifndef BLOAD_GRANULE_UNPACK
#define BLOAD_GRANULE_UNPACK 1  // 0: whole-plan unpack of these frames stays on the register path (to compare)
#endif
#ifndef BLOAD_GRANULE_MAX_FRAME
#define BLOAD_GRANULE_MAX_FRAME 3
#endif
// Pack of frames of 1 to 3 bytes (per-token masks, 16-bit ids or scalars) in runs beyond the 2- and 1-byte walks and up
// to 4 KB on average: k24_pack_granules instead of the register path.  Measured on B200 (TB/s, granules against the
// register path; about 1.5 GB per case): token lengths, 1-byte frames (870-byte runs) 3.70 against 2.52, 2-byte frames
// (1.7 KB) 4.43 against 3.66, 3-byte frames (2.6 KB) 4.56 against 4.28; beyond that the register path is as fast
// or faster: 6-byte frames (5.2 KB) 4.96 against 4.93, 10-byte (8.7 KB) 5.21 against 5.42, 30-byte (26 KB) 5.54 against
// 6.00; 30-byte frames in heavy-tailed 1.7 KB runs 2.98 against 3.07, 250-byte frames in 5.5 KB clips 4.47 against 4.28.
// Whole-plan unpack of the same frames along the ragged side (k25_unpack_granules), same cases: 3.67 against 3.23, 4.71
// against 4.19, 5.02 against 4.6.
// In short runs the word-wise walks stay (granules against them, pack / unpack): 6-byte frames in 346-byte runs 1.44 /
// 1.83 against 2.87 / 3.02, 3-byte frames in 173-byte runs 1.01 / 1.32 against 1.49 / 1.60, 30-byte frames in 663-byte
// runs 2.09 / 2.60 against 3.19 / 3.35: a granule that holds a run's end is moved byte by byte.
constexpr int64_t kGranuleMaxRun = BLOAD_GRANULE_MAX_RUN, kGranuleMaxFrame = BLOAD_GRANULE_MAX_FRAME;
inline bool walks_unstaged(int64_t frame_bytes, int64_t mean_run, bool unpack)
{
    if (frame_bytes % 8 == 0) return mean_run <= kStagedMaxRunBytes;
    if (frame_bytes % 4 == 0) return false;
    if (!BLOAD_ODD_WALKS) return false;
    if (frame_bytes % 2 == 0) return mean_run <= (unpack ? 1024 : 1536);
    return mean_run <= 384;
}

// ------------------------------------------------------------------------------------------------
// Measurement variant, compiled only with -DBLOAD_BULK_COPY=1 (never in the default library): the large-frame path
// through the bulk-copy engine instead of registers.  Frames whose size is a multiple of 16 bytes; a warp owns a ring
// of shared-memory stages, each the image of one sub-tile of the dense side.  Pack: every run piece of the sub-tile
// arrives by one cp.async.bulk (global -> shared, completion counted in bytes on the stage's mbarrier), padding is
// written with shared stores, the sub-tile leaves with ONE bulk store.  Unpack: the occupied part of the sub-tile
// arrives by ONE bulk load and leaves with one bulk store per run piece.  It exists so that the comparison "bulk
// engine against register path" can be repeated from this source; on B200 the register path is faster (see the
// measurements next to launch_copy).  The only waits are on the warp's own mbarriers and bulk groups; the mbarrier
// wait gives up after a fixed number of polls, counts the event (bload_bulk_copy_timeouts) and lets the warp finish.
#if BLOAD_BULK_COPY
#ifndef BLOAD_BULK_BYTES
#define BLOAD_BULK_BYTES 8192
#endif
#ifndef BLOAD_BULK_WARPS
#define BLOAD_BULK_WARPS 4
#endif
#ifndef BLOAD_BULK_STAGES
#define BLOAD_BULK_STAGES 3
#endif
static __device__ unsigned int g_bulk_timeouts;

__device__ __forceinline__ void mbar_init(uint32_t bar)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* g, uint32_t bytes, uint32_t bar)
{
    if (!BLOAD_MAY_READ(g, bytes)) return;
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_dst), "l"(g), "r"(bytes), "r"(bar) : "memory");
}
// true when the phase with this parity has completed; gives up after kPolls polls
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    constexpr int kPolls = 1 << 22;
    for (int i = 0; i < kPolls; ++i) {
        uint32_t done;
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (done) return true;
    }
    atomicAdd(&g_bulk_timeouts, 1u);
    return false;
}

template <bool UNPACK>
__global__ void __launch_bounds__(BLOAD_BULK_WARPS * 32) k7b_copy_bulk(PlanView pv, int32_t t_block, int64_t frame_bytes,
                                                                      int64_t block_begin, int64_t block_count,
                                                                      const uint8_t* __restrict__ src_base,
                                                                      uint8_t* __restrict__ dst_base, int64_t subs_per_block,
                                                                      uint8_t pad)
{
    constexpr int NST = BLOAD_BULK_STAGES, kBytes = BLOAD_BULK_BYTES, kWarps = BLOAD_BULK_WARPS;
    extern __shared__ __align__(128) uint8_t stage_mem[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint8_t* my_stages = stage_mem + (size_t)warp * NST * kBytes;
    const uint32_t my_bars = smem_addr(stage_mem + (size_t)kWarps * NST * kBytes) + (uint32_t)warp * NST * 8;
    if (lane == 0) {
        for (int i = 0; i < NST; ++i) mbar_init(my_bars + 8 * i);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const int64_t warps = (int64_t)gridDim.x * kWarps;
    const int64_t items = block_count * subs_per_block;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t n_blocks = pv.hdr->n_blocks;
    const uint32_t p4 = 0x01010101u * pad;
    uint32_t parity_bits = 0;  // bit i: parity of the phase stage i's barrier is in

    // what the second phase of an item needs
    struct Pending { int64_t dense_off; int64_t b; int lo; int nbytes; int valid; int k; int k1; int fill; bool wait; };
    Pending prev{};
    bool have_prev = false, alive = true;
    int s = 0, s_prev = 0;

    // second phase: the loads of the item have landed in `stage`
    auto complete = [&](const Pending& it, uint8_t* stage, int st_idx) {
        if (it.wait) {
            bool ok = true;
            if (lane == 0) ok = mbar_wait(my_bars + 8 * st_idx, (parity_bits >> st_idx) & 1u);
            ok = __shfl_sync(kFull, ok, 0);
            parity_bits ^= 1u << st_idx;
            if (!ok) { alive = false; return; }
        }
        fence_proxy_async();  // shared stores of padding before the bulk store reads them
        __syncwarp();
        if (!UNPACK) {
            if (lane == 0) bulk_store(dst_base + it.dense_off, smem_addr(stage), (uint32_t)it.nbytes);
        } else if (it.valid > 0) {
            // one bulk store per run piece of the occupied part
            int k = it.k, kw = it.k;
            int w_st = (kw + lane < it.k1) ? pv.seg_start[kw + lane] : it.fill;
            int64_t w_src = (kw + lane < it.k1) ? pv.seg_src[kw + lane] : 0;
            int64_t cur = it.lo;
            const int64_t hi = (int64_t)it.lo + it.valid;
            while (cur < hi && k < it.k1) {
                if (k - kw == 31) {
                    kw = k;
                    w_st = (kw + lane < it.k1) ? pv.seg_start[kw + lane] : it.fill;
                    w_src = (kw + lane < it.k1) ? pv.seg_src[kw + lane] : 0;
                }
                const int st = __shfl_sync(kFull, w_st, k - kw);
                const int nx = __shfl_sync(kFull, w_st, k - kw + 1);
                const int64_t src_frame = __shfl_sync(kFull, w_src, k - kw);
                const int64_t pe = min((int64_t)nx * frame_bytes, hi);
                const int64_t rag = src_frame * frame_bytes + (cur - (int64_t)st * frame_bytes);
                if (lane == 0) bulk_store(dst_base + rag, smem_addr(stage) + (uint32_t)(cur - it.lo), (uint32_t)(pe - cur));
                cur = pe;
                ++k;
            }
        }
        if (lane == 0) bulk_commit();
    };

    for (int64_t item = (int64_t)blockIdx.x * kWarps + warp; item < items && alive; item += warps) {
        const int64_t q = item / subs_per_block;
        Pending it{};
        it.lo = (int)((item - q * subs_per_block) * kBytes);
        it.nbytes = (int)min((int64_t)kBytes, block_bytes - it.lo);
        it.b = block_begin + q;
        it.dense_off = q * block_bytes + it.lo;
        int k0 = 0;
        if (it.b < n_blocks) { k0 = pv.block_seg_begin[it.b]; it.k1 = pv.block_seg_begin[it.b + 1]; it.fill = pv.block_fill[it.b]; }
        const int64_t fill_bytes = (int64_t)it.fill * frame_bytes;
        it.valid = it.lo < fill_bytes ? (int)min((int64_t)it.nbytes, fill_bytes - it.lo) : 0;
        it.wait = it.valid > 0;
        it.k = it.valid > 0 ? warp_find_segment(pv.seg_start, k0, it.k1, (int)(it.lo / frame_bytes), lane) : k0;
        uint8_t* stage = my_stages + (size_t)s * kBytes;
        const uint32_t sa = smem_addr(stage), bar = my_bars + 8 * s;
        if (lane == 0) bulk_wait_read<NST - 2>();  // the stores that last read this stage have finished reading
        __syncwarp();
        if (it.valid > 0) {
            if (lane == 0) mbar_expect_tx(bar, (uint32_t)it.valid);
            if (UNPACK) {
                if (lane == 0) bulk_load(sa, src_base + it.dense_off, (uint32_t)it.valid, bar);
            } else {
                int k = it.k, kw = it.k;
                int w_st = (kw + lane < it.k1) ? pv.seg_start[kw + lane] : it.fill;
                int64_t w_src = (kw + lane < it.k1) ? pv.seg_src[kw + lane] : 0;
                int64_t cur = it.lo;
                const int64_t hi = (int64_t)it.lo + it.valid;
                while (cur < hi && k < it.k1) {
                    if (k - kw == 31) {
                        kw = k;
                        w_st = (kw + lane < it.k1) ? pv.seg_start[kw + lane] : it.fill;
                        w_src = (kw + lane < it.k1) ? pv.seg_src[kw + lane] : 0;
                    }
                    const int st = __shfl_sync(kFull, w_st, k - kw);
                    const int nx = __shfl_sync(kFull, w_st, k - kw + 1);
                    const int64_t src_frame = __shfl_sync(kFull, w_src, k - kw);
                    const int64_t pe = min((int64_t)nx * frame_bytes, hi);
                    const int64_t rag = src_frame * frame_bytes + (cur - (int64_t)st * frame_bytes);
                    if (lane == 0) bulk_load(sa + (uint32_t)(cur - it.lo), src_base + rag, (uint32_t)(pe - cur), bar);
                    cur = pe;
                    ++k;
                }
            }
        }
        if (!UNPACK)  // padding behind the frames (valid and nbytes are multiples of 16 here)
            for (int o = it.valid + 16 * lane; o < it.nbytes; o += 512) *reinterpret_cast<uint4*>(stage + o) = make_uint4(p4, p4, p4, p4);
        if (have_prev) complete(prev, my_stages + (size_t)s_prev * kBytes, s_prev);
        prev = it; have_prev = true; s_prev = s;
        s = (s + 1 == NST) ? 0 : s + 1;
    }
    if (have_prev && alive) complete(prev, my_stages + (size_t)s_prev * kBytes, s_prev);
    __syncwarp();
    if (lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // the warp's own stores are complete
}
#endif  // BLOAD_BULK_COPY

}  // namespace

// Pack and per-slot metadata of a few blocks of small word-sized frames in ONE launch (see k10_pack_contig<true>);
// false when the call does not suit the staged pack kernel or is large enough for two full-speed launches.
bool staged_pack_with_metadata(const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                               int64_t block_count, const uint8_t* store, uint8_t* dense, int32_t* seq_id, int32_t* pos,
                               uint8_t* reset, uint8_t* valid, int64_t ragged_bytes, uint8_t pad_byte, cudaStream_t st,
                               int64_t n, cudaError_t* err)
{
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    constexpr int64_t kMaxFusedSlots = 1 << 22;  // beyond this the metadata kernel's own launch shape is faster
    if (!(frame_bytes % 4 == 0 && n > 0 && n < 0x7fffff00LL && ragged_bytes / n <= kStagedMaxRunBytes && block_bytes < (1LL << 30) &&
          block_count * t_block <= kMaxFusedSlots))
        return false;
    const bool by_words = runs_are_short(ragged_bytes, n, frame_bytes);  // very short runs: the word-wise kernel
    const StagedShape Cfg = !by_words ? shape_of<StageCfg<false>>() : frame_bytes % 16 == 0 ? shape_of<ShortCfg<16>>() : shape_of<ShortCfg<4>>();
    const size_t smem = (size_t)Cfg.kWarps * Cfg.kStages * Cfg.kBytes + 16 + (by_words ? (size_t)Cfg.kWarps * kShortWindowBytes : 0);
    using PackKernel = void (*)(PlanView, int32_t, int32_t, int64_t, int64_t, const uint8_t*, uint8_t*, int64_t, int64_t, int64_t, uint8_t, MetaOut);
    const PackKernel kernel = !by_words ? k10_pack_contig<true>
                              : frame_bytes % 16 == 0 ? k17_pack_short_runs<true, 16>
                              : frame_bytes % 8 == 0 ? k17_pack_short_runs<true, 8> : k17_pack_short_runs<true, 4>;
    *err = opt_in_shared_memory(kernel, (int)smem);
    if (*err != cudaSuccess) return true;
    const DeviceInfo di = device_info();
    const int per_sm = (int)(di.smem_per_sm / (smem + 1024));
    const int64_t total = block_count * block_bytes;
    const int64_t tiles = (total + Cfg.kBytes - 1) / Cfg.kBytes;
    const int64_t max_warps = (int64_t)di.sm_count * per_sm * Cfg.kWarps;
    int64_t tpw = (tiles + max_warps - 1) / max_warps;
    if (tpw > (by_words ? kShortChunkTiles : kPackChunkTiles)) tpw = by_words ? kShortChunkTiles : kPackChunkTiles;
    int64_t warps = (tiles + tpw - 1) / tpw;
    if (warps > max_warps) warps = max_warps;
    auto al = [](const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; };
    MetaOut mo;
    mo.seq_id = seq_id; mo.pos = pos; mo.reset = reset; mo.valid = valid;
    mo.pack_ctas = (uint32_t)((warps + Cfg.kWarps - 1) / Cfg.kWarps);
    mo.chunks_per_block = (int32_t)((t_block + Cfg.kWarps * 128 - 1) / (Cfg.kWarps * 128));
    mo.vec = t_block % 4 == 0 && al(seq_id, 16) && al(pos, 16) && al(reset, 4) && al(valid, 4);
    const int64_t grid = (int64_t)mo.pack_ctas + block_count * mo.chunks_per_block;
    count_launches(1);
    {
        [[maybe_unused]] const size_t slots = (size_t)block_count * (size_t)t_block;
        BLOAD_DBG_EXPECT(st, dbg::kPackContig, {{store, (size_t)ragged_bytes}},
                         {{dense, (size_t)(block_count * block_bytes)}, {seq_id, 4 * slots}, {pos, 4 * slots}, {reset, slots}, {valid, slots}});
    }
    note_copy_kernel(kCallPack, by_words ? "k17_pack_short_runs<metadata>" : "k10_pack_contig<metadata>");
    kernel<<<(unsigned)grid, Cfg.kWarps * 32, smem, st>>>(pv, (int32_t)n, t_block, frame_bytes, block_begin, store, dense, tiles, tpw,
                                                         total, pad_byte, mo);
    *err = cudaPeekAtLastError();
    return true;
}

cudaError_t launch_copy(bool unpack, const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                        int64_t block_count, const uint8_t* ragged_in, uint8_t* dense, uint8_t* ragged_out,
                        int64_t ragged_bytes, uint8_t pad_byte, cudaStream_t st, int64_t n, int64_t n_blocks, bool gaps,
                        bool beside_previous)
{
    if (block_count == 0) return cudaSuccess;
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    count_launches(1);
    if (unpack) BLOAD_DBG_EXPECT(st, dbg::kCopy, {{dense, (size_t)(block_count * block_bytes)}}, {{ragged_out, (size_t)ragged_bytes}});
    else BLOAD_DBG_EXPECT(st, dbg::kCopy, {{ragged_in, (size_t)ragged_bytes}}, {{dense, (size_t)(block_count * block_bytes)}});
    // Which family moves the frames (measured cross-overs beside walks_unstaged and runs_are_short):
    //   unstaged word-wise walks   frames that are multiples of 8 bytes in runs of at most 16 KB on average; frames that
    //                              are not multiples of 4 bytes in short runs; 4-byte-word frames in short runs when a
    //                              block sub-range is unpacked
    //   staged, word by word       frames that are multiples of 4 (not 8) bytes in runs of at most 768 bytes
    //   staged, run by run         the other frames that are multiples of 4 bytes, in runs of at most 16 KB
    //   granules of 16 bytes       pack and whole-plan unpack of frames of 1 to 3 bytes in runs beyond the walks, up to
    //                              4 KB on average
    //   register path              everything else
    // (the staged kernels and the walks index windows of 32 runs past a 32-bit position in the segment list)
    const bool indexable = n > 0 && n < 0x7fffff00LL && block_bytes < (1LL << 30);
    const int64_t mean_run = n > 0 ? ragged_bytes / n : 0;
    const bool short_runs = frame_bytes % 4 == 0 && indexable && mean_run <= kStagedMaxRunBytes;
    const bool whole_plan = unpack && !gaps && block_begin == 0 && block_count >= n_blocks && ragged_bytes > 0;
    const bool by_words = short_runs && runs_are_short(ragged_bytes, n, frame_bytes);
    if (indexable && (walks_unstaged(frame_bytes, mean_run, unpack) || (by_words && unpack && !whole_plan))) {
        const int64_t cap = (int64_t)device_info().sm_count * 32;
        if (whole_plan) {  // along the ragged side, which is contiguous and written completely
            const WalkRaggedKernel kernel = walk_ragged_kernel_for(frame_bytes);
            const int piece = walk_piece_bytes(ragged_bytes, device_info().sm_count);
            const int64_t want = ((ragged_bytes + piece - 1) / piece + 7) / 8;
            kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(pv, (int32_t)n, t_block, frame_bytes, ragged_bytes / frame_bytes,
                                                                        dense, ragged_out, piece);
            note_copy_kernel(kCallUnpack, "k21_unpack_walk_ragged");
            return cudaPeekAtLastError();
        }
        const WalkKernel kernel = unpack ? walk_kernel_for<false>(frame_bytes) : walk_kernel_for<true>(frame_bytes);
        const int64_t total = block_count * block_bytes;
        const int piece = walk_piece_bytes(total, device_info().sm_count);
        const int64_t want = ((total + piece - 1) / piece + 7) / 8;
        kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(pv, (int32_t)n, t_block, frame_bytes, block_begin,
                                                                    unpack ? dense : ragged_in, unpack ? ragged_out : dense, total, pad_byte, piece);
        note_copy_kernel(unpack ? kCallUnpack : kCallPack, unpack ? "k19_unpack_walk_dense" : "k19_pack_walk_dense");
        return cudaPeekAtLastError();
    }
    // pack of small word-sized frames: contiguous ranges of dense sub-tiles per warp
    if (!unpack && short_runs) {
        // (frames that are multiples of 8 bytes went to the walks above: words of 4 bytes here)
        const StagedShape Cfg = by_words ? shape_of<ShortCfg<4>>() : shape_of<StageCfg<false>>();
        const size_t smem = (size_t)Cfg.kWarps * Cfg.kStages * Cfg.kBytes + 16 + (by_words ? (size_t)Cfg.kWarps * kShortWindowBytes : 0);
        const DeviceInfo di = device_info();
        const int per_sm = (int)(di.smem_per_sm / (smem + 1024));
        using PackKernel = void (*)(PlanView, int32_t, int32_t, int64_t, int64_t, const uint8_t*, uint8_t*, int64_t, int64_t, int64_t, uint8_t, MetaOut);
        const PackKernel kernel = by_words ? k17_pack_short_runs<false, 4> : k10_pack_contig<false>;
        cudaError_t e = opt_in_shared_memory(kernel, (int)smem);
        if (e != cudaSuccess) return e;
        const int64_t total = block_count * block_bytes;
        const int64_t tiles = (total + Cfg.kBytes - 1) / Cfg.kBytes;  // of the dense side as one array: blocks begin anywhere
        const int64_t max_warps = (int64_t)di.sm_count * per_sm * Cfg.kWarps;
        int64_t tpw = (tiles + max_warps - 1) / max_warps;
        if (tpw > (by_words ? kShortChunkTiles : kPackChunkTiles)) tpw = by_words ? kShortChunkTiles : kPackChunkTiles;  // grid-strided beyond
        int64_t warps = (tiles + tpw - 1) / tpw;
        if (warps > max_warps) warps = max_warps;
        const unsigned grid = (unsigned)((warps + Cfg.kWarps - 1) / Cfg.kWarps);
        kernel<<<grid, Cfg.kWarps * 32, smem, st>>>(pv, (int32_t)n, t_block, frame_bytes, block_begin, ragged_in, dense, tiles, tpw, total,
                                                   pad_byte, MetaOut{});
        note_copy_kernel(kCallPack, by_words ? "k17_pack_short_runs" : "k10_pack_contig");
        return cudaPeekAtLastError();
    }
    // whole-plan unpack of small word-sized frames: tile the (contiguous, fully written) ragged side
    // (not when frames between the plan's sequences belong to nobody: this path writes the whole ragged buffer)
    if (whole_plan && short_runs) {
        const DeviceInfo di = device_info();
        const StagedShape c = by_words ? shape_of<ShortCfg<4>>() : shape_of<StageCfg<false>>();
        const size_t smem = (size_t)c.kWarps * c.kStages * c.kBytes + 16 + (by_words ? (size_t)c.kWarps * kShortWindowBytes : 0);
        const int64_t tiles = (ragged_bytes + c.kBytes - 1) / c.kBytes;
        const int per_sm = (int)(di.smem_per_sm / (smem + 1024));
        const int64_t max_warps = (int64_t)di.sm_count * per_sm * c.kWarps;
        const int64_t tpw = (tiles + max_warps - 1) / max_warps;  // contiguous sub-tiles per warp
        const int64_t warps = (tiles + tpw - 1) / tpw;
        const unsigned grid = (unsigned)((warps + c.kWarps - 1) / c.kWarps);
        // (the word-wise kernel keeps 32-bit positions inside a warp's range)
        const bool words = by_words && tpw * c.kBytes < (1LL << 30);
        using UnpackKernel = void (*)(PlanView, int32_t, int32_t, int64_t, int64_t, const uint8_t*, uint8_t*, int64_t, int64_t);
        const UnpackKernel kernel = words ? k18_unpack_short_runs<4> : k9_unpack_ragged;
        if (words || !by_words) {
            cudaError_t e = opt_in_shared_memory(kernel, (int)smem);
            if (e != cudaSuccess) return e;
            kernel<<<grid, c.kWarps * 32, smem, st>>>(pv, (int32_t)n, t_block, frame_bytes, ragged_bytes / frame_bytes, dense, ragged_out,
                                                    tiles, tpw);
            note_copy_kernel(kCallUnpack, words ? "k18_unpack_short_runs" : "k9_unpack_ragged");
            return cudaPeekAtLastError();
        }
    }
    // block sub-ranges of small word-sized frames, unpack direction: staged kernel over the dense side
    if (unpack && short_runs && block_bytes % 16 == 0) {
        using Cfg = StageCfg<true>;
        const int64_t spb = (block_bytes + Cfg::kBytes - 1) / Cfg::kBytes;
        const int64_t gpb = (spb + Cfg::kGroup - 1) / Cfg::kGroup;  // groups of sub-tiles per block
        const size_t smem = (size_t)Cfg::kWarps * Cfg::kStages * Cfg::kBytes + 16;  // 16 spare bytes: see warp_scatter
        const DeviceInfo di = device_info();
        const int per_sm = (int)(di.smem_per_sm / (smem + 1024));
        cudaError_t e = opt_in_shared_memory(k8_unpack_staged, (int)smem);
        if (e != cudaSuccess) return e;
        // 32-bit group arithmetic on the device: at most 2^31 - 1 groups per launch
        const int64_t max_blocks = 0x7fffffffLL / gpb;
        for (int64_t done = 0; done < block_count; done += max_blocks) {
            const int64_t cnt = block_count - done < max_blocks ? block_count - done : max_blocks;
            const int64_t groups = cnt * gpb;
            const int64_t want = (groups + Cfg::kWarps - 1) / Cfg::kWarps;
            const unsigned grid = (unsigned)(want < (int64_t)di.sm_count * per_sm ? want : (int64_t)di.sm_count * per_sm);
            k8_unpack_staged<<<grid, Cfg::kWarps * 32, smem, st>>>(pv, t_block, frame_bytes, block_begin + done, (uint32_t)groups,
                                                                 dense + done * block_bytes, ragged_out, (uint32_t)gpb, pad_byte);
        }
        note_copy_kernel(kCallUnpack, "k8_unpack_staged");
        return cudaPeekAtLastError();
    }
    // whole-plan unpack of the same frames, along the ragged side
    if (BLOAD_GRANULE_UNPACK && whole_plan && indexable && frame_bytes % 4 != 0 && frame_bytes <= kGranuleMaxFrame && mean_run <= kGranuleMaxRun) {
        const int64_t cap = (int64_t)device_info().sm_count * 32;
        const int piece = walk_piece_bytes(ragged_bytes, device_info().sm_count);
        const int64_t want = ((ragged_bytes + piece - 1) / piece + 7) / 8;
        k25_unpack_granules<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(pv, (int32_t)n, t_block, frame_bytes, ragged_bytes / frame_bytes,
                                                                                  dense, ragged_out, block_count * block_bytes, piece);
        note_copy_kernel(kCallUnpack, "k25_unpack_granules");
        return cudaPeekAtLastError();
    }
    // pack of frames that are not multiples of 4 bytes, in runs beyond the 2- and 1-byte walks: granules of 16 bytes
    if (!unpack && indexable && frame_bytes % 4 != 0 && frame_bytes <= kGranuleMaxFrame && mean_run <= kGranuleMaxRun) {
        const int64_t cap = (int64_t)device_info().sm_count * 32;
        const int64_t total = block_count * block_bytes;
        const int piece = walk_piece_bytes(total, device_info().sm_count);
        const int64_t want = ((total + piece - 1) / piece + 7) / 8;
        k24_pack_granules<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(pv, (int32_t)n, t_block, frame_bytes, block_begin, ragged_in,
                                                                                dense, total, ragged_bytes, pad_byte, piece);
        note_copy_kernel(kCallPack, "k24_pack_granules");
        return cudaPeekAtLastError();
    }
#if BLOAD_BULK_COPY
    if (frame_bytes % 16 == 0) {  // the measurement variant through the bulk-copy engine
        constexpr int kB = BLOAD_BULK_BYTES, kW = BLOAD_BULK_WARPS, kS = BLOAD_BULK_STAGES;
        const size_t smem = (size_t)kW * kS * kB + (size_t)kW * kS * 8;
        const DeviceInfo di = device_info();
        const int per_sm = (int)(di.smem_per_sm / (smem + 1024));
        const int64_t spb_b = (block_bytes + kB - 1) / kB;
        const int64_t want_b = (block_count * spb_b + kW - 1) / kW, cap = (int64_t)di.sm_count * (per_sm > 0 ? per_sm : 1);
        const unsigned grid_b = (unsigned)(want_b < cap ? want_b : cap);
        cudaError_t e = opt_in_shared_memory(unpack ? k7b_copy_bulk<true> : k7b_copy_bulk<false>, (int)smem);
        if (e != cudaSuccess) return e;
        note_copy_kernel(unpack ? kCallUnpack : kCallPack, unpack ? "k7b_copy_bulk<unpack>" : "k7b_copy_bulk<pack>");
        if (unpack)
            k7b_copy_bulk<true><<<grid_b, kW * 32, smem, st>>>(pv, t_block, frame_bytes, block_begin, block_count, dense, ragged_out,
                                                              spb_b, pad_byte);
        else
            k7b_copy_bulk<false><<<grid_b, kW * 32, smem, st>>>(pv, t_block, frame_bytes, block_begin, block_count, ragged_in, dense,
                                                               spb_b, pad_byte);
        return cudaPeekAtLastError();
    }
#endif
    note_copy_kernel(unpack ? kCallUnpack : kCallPack, unpack ? "k7_copy<unpack>" : "k7_copy<pack>");
    const int64_t sub = 16384;
    const int64_t spb = (block_bytes + sub - 1) / sub;
    const int64_t items = block_count * spb;
    const int64_t want = (items + 7) / 8;
    // one sub-tile per warp, as many CTAs as that takes: measured 1 % faster than a persistent grid of 148 x 8
    // CTAs (6.63 / 6.65 against 6.54 / 6.59 TB/s) and kinder to small kernels of other streams, which then
    // find free slots between short-lived CTAs; the grid-stride loop only matters beyond 2^31 - 1 CTAs
    const unsigned grid = (unsigned)(want < 0x7fffffffLL ? want : 0x7fffffffLL);
    if (unpack)
        k7_copy<true><<<grid, 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count, dense, ragged_out,
                                             block_count * block_bytes, sub, spb, pad_byte, nullptr, block_begin);
    else if (beside_previous && !dbg::kChecked) {
        // measured on B200, per-batch calls (dense blocks + metadata, two launches): 8 blocks of 41 MB 112.0 -> 105.5 us
        // per call (107.4 -> 102.9 replayed from a graph), 4 blocks of 135 MB 168.8 -> 163.2 us (164.4 -> 160.2)
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3(grid); cfg.blockDim = dim3(256); cfg.dynamicSmemBytes = 0; cfg.stream = st;
        cudaLaunchAttribute at[1];
        at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        at[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = at; cfg.numAttrs = 1;
        const int32_t* no_range = nullptr;
        return cudaLaunchKernelEx(&cfg, k7_copy<false>, pv, t_block, frame_bytes, block_begin, block_count, ragged_in,
                                  dense, ragged_bytes, sub, spb, pad_byte, no_range, block_begin);
    } else
        k7_copy<false><<<grid, 256, 0, st>>>(pv, t_block, frame_bytes, block_begin, block_count, ragged_in, dense,
                                              ragged_bytes, sub, spb, pad_byte, nullptr, block_begin);
    return cudaPeekAtLastError();
}

// Register-path copy of the blocks named by a device-side range (see k7_copy): a fixed grid whose warps loop, because
// the host does not know how many blocks the range holds.  The dense buffer starts at block 0.
cudaError_t launch_copy_range(bool unpack, const PlanView& pv, int32_t t_block, int64_t frame_bytes, const uint8_t* src,
                              uint8_t* dst, int64_t src_total_bytes, uint8_t pad_byte, const int32_t* d_range,
                              cudaStream_t st)
{
    const int64_t block_bytes = (int64_t)t_block * frame_bytes;
    const int64_t sub = 16384;
    const int64_t spb = (block_bytes + sub - 1) / sub;
    // many short-lived CTAs rather than a few long ones: the next chunk of the fill rule (one CTA on the other stream)
    // starts as soon as any CTA of this launch retires; a chunk holds some thousand sub-tiles, about one per warp
    const unsigned grid = (unsigned)device_info().sm_count * 3 * 16;  // (2 to 32 rounds of resident CTAs measured alike)
    count_launches(1);
    BLOAD_DBG_UNCHECKED(st);  // runs beside launches of another stream, on a block range only the device knows
    if (unpack)
        k7_copy<true><<<grid, 256, kBesideChainSmemBytes, st>>>(pv, t_block, frame_bytes, 0, 0, src, dst, src_total_bytes, sub, spb,
                                                                pad_byte, d_range, 0);
    else
        k7_copy<false><<<grid, 256, kBesideChainSmemBytes, st>>>(pv, t_block, frame_bytes, 0, 0, src, dst, src_total_bytes, sub, spb,
                                                                 pad_byte, d_range, 0);
    return cudaPeekAtLastError();
}


// mbarrier waits that gave up in the bulk-copy measurement variant since the library was loaded (0 in the default build)
unsigned int bulk_copy_timeouts()
{
#if BLOAD_BULK_COPY
    unsigned int v = 0;
    if (cudaDeviceSynchronize() != cudaSuccess || cudaMemcpyFromSymbol(&v, g_bulk_timeouts, sizeof v) != cudaSuccess) {
        (void)cudaGetLastError();
        return ~0u;
    }
    return v;
#else
    return 0;
#endif
}

}  // namespace bload

// Best fit decreasing (policy 2): a deterministic comparison strategy, NOT the paper's random rule.
//
// Sequences are taken in decreasing order of length (the reverse of the sorted L_dict array).  Each one
// goes to the open block whose free room is the smallest that still holds it -- among blocks with equal
// room, the one that has had that room longest -- or opens a new block.  Only the multiset of free rooms
// steers these decisions, so the sequential part keeps no block identities at all:
//   1. chain kernel (one warp): per room value a count of open blocks and a two-level bitmap of the
//      non-empty rooms in shared memory; per item a successor query ("smallest non-empty room >= length"),
//      two count updates, and a record {room taken (0 = new block), room left};
//   2. parallel passes: the i-th item that takes a block of room r continues the i-th item that left a
//      block with room r (first in, first out), which two stable sorts by room turn into a predecessor
//      pointer per item; pointer doubling resolves every item to the item that opened its block; new blocks
//      are numbered in opening order; a stable sort by block gives the segment list in placement order.
// The start slot of an item needs no chain at all: it is t_block minus the room it took.
#include <limits.h>

#include "bload_internal.cuh"

namespace bload {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr unsigned long long kNoBad = ULLONG_MAX;

// ---- 1. the chain: one warp, all lanes compute the same scalars, lane 0 writes ----
__global__ void __launch_bounds__(256, 1) kb_chain(const PlanHeader* hdr, const uint64_t* __restrict__ sorted_key,
                                                   int2* __restrict__ rec, int32_t n, int32_t L)
{
    extern __shared__ __align__(16) int32_t sm[];
    // rooms 1..L map to bits 0..L-1 of B2
    uint32_t* B2 = reinterpret_cast<uint32_t*>(sm);        // [1024] bit set: some open block has that room
    int2* ring = reinterpret_cast<int2*>(sm + 1024);       // [32] records of the last items
    int32_t* cnt = sm + 1024 + 64;                         // [L] open blocks per room
    if (hdr->first_bad != kNoBad) return;
    for (int i = threadIdx.x; i < 1024; i += blockDim.x) B2[i] = 0;
    for (int i = threadIdx.x; i < L; i += blockDim.x) cnt[i] = 0;
    __syncthreads();
    if (threadIdx.x >= 32) return;
    const int lane = threadIdx.x;
    uint32_t b1 = 0;                                       // lane i: which of the words 32i .. 32i+31 of B2 are non-zero
    // lengths of 32 items at a time, one per lane (item t is sorted position n-1-t), the next 32 prefetched
    auto len_of = [&](int t) { return t < n ? (int)(sorted_key[n - 1 - t] >> 32) : 1; };
    int len_cur = len_of(lane), len_nxt = len_of(32 + lane);
    for (int t = 0; t < n; ++t) {
        const int l = __shfl_sync(kFull, len_cur, t & 31);
        const int q = l - 1, w0 = q >> 5;
        int ridx = -1;                                     // bit index of the room taken, -1: open a new block
        const uint32_t x = B2[w0] & (0xffffffffu << (q & 31));
        if (x) {
            ridx = (w0 << 5) + __ffs(x) - 1;
        } else {                                           // next non-empty word after w0, if any
            const int lw = (w0 + 1) >> 5, lb = (w0 + 1) & 31;
            const uint32_t mine = lane > lw ? b1 : (lane == lw ? (b1 & (0xffffffffu << lb)) : 0u);
            const uint32_t bal = __ballot_sync(kFull, mine != 0);
            if (bal) {
                const int f = __ffs(bal) - 1;
                const uint32_t wf = __shfl_sync(kFull, mine, f);
                const int w = (f << 5) + __ffs(wf) - 1;
                ridx = (w << 5) + __ffs(B2[w]) - 1;
            }
        }
        if (ridx >= 0) {                                   // one block less with that room
            const int c = cnt[ridx] - 1, w = ridx >> 5;
            const uint32_t word = c == 0 ? (B2[w] & ~(1u << (ridx & 31))) : B2[w];
            if (lane == 0) { cnt[ridx] = c; B2[w] = word; }
            if (word == 0 && lane == (w >> 5)) b1 &= ~(1u << (w & 31));
        }
        __syncwarp();
        const int left = (ridx >= 0 ? ridx + 1 : L) - l;   // room left in the block after this item
        if (left > 0) {                                    // one block more with the room that is left
            const int idx = left - 1, w = idx >> 5;
            const int c = cnt[idx];
            const uint32_t word = B2[w] | (1u << (idx & 31));
            if (lane == 0) { cnt[idx] = c + 1; B2[w] = word; }
            if (lane == (w >> 5)) b1 |= 1u << (w & 31);
        }
        if (lane == 0) ring[t & 31] = make_int2(ridx + 1, left);
        __syncwarp();
        if (((t + 1) & 31) == 0) {
            rec[t - 31 + lane] = ring[lane];
            len_cur = len_nxt;
            len_nxt = len_of(t + 33 + lane);
            __syncwarp();
        }
    }
    if (lane < (n & 31)) rec[(n & ~31) + lane] = ring[lane];
}

// ---- 2. parallel passes ----
__global__ void __launch_bounds__(256) kb_event_keys(const PlanHeader* hdr, const int2* __restrict__ rec, int64_t n,
                                                     uint64_t* __restrict__ key, int32_t* __restrict__ id, int which)
{
    if (hdr->first_bad != kNoBad) return;
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= n) return;
    const int2 r = rec[t];
    key[t] = (uint64_t)(uint32_t)(which ? r.y : r.x) << 32;   // room in the high word, as the bucket kernel expects
    id[t] = (int32_t)t;
}

// predecessor of every item: the item after which it was appended to its block (itself if it opened the block),
// and the block number of the items that opened one (their rank among such items, which the stable sort kept)
__global__ void __launch_bounds__(256) kb_pred(const PlanHeader* hdr, const uint64_t* __restrict__ take_key,
                                               const int32_t* __restrict__ take_item, const int32_t* __restrict__ take_end,
                                               const int32_t* __restrict__ put_item, const int32_t* __restrict__ put_end,
                                               int64_t n, int32_t* __restrict__ pred, int32_t* __restrict__ blk)
{
    if (hdr->first_bad != kNoBad) return;
    const int64_t p = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (p >= n) return;
    const int r = (int)(take_key[p] >> 32);
    const int t = take_item[p];
    if (r == 0) { pred[t] = t; blk[t] = (int32_t)p; return; }     // the p-th new block
    const int rank = (int)(p - take_end[r - 1]);                     // p-th item that took a block of room r
    pred[t] = put_item[put_end[r - 1] + rank];                       // continues the rank-th item that left room r
    blk[t] = -1;
}

__global__ void __launch_bounds__(256) kb_jump(const PlanHeader* hdr, const int32_t* __restrict__ in, int32_t* __restrict__ out, int64_t n)
{
    if (hdr->first_bad != kNoBad) return;
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t < n) out[t] = in[in[t]];
}

__global__ void __launch_bounds__(256) kb_block_keys(const PlanHeader* hdr, const int32_t* __restrict__ root, int32_t* __restrict__ blk,
                                                     int64_t n, uint64_t* __restrict__ key, int32_t* __restrict__ id)
{
    if (hdr->first_bad != kNoBad) return;
    const int64_t t = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (t >= n) return;
    const int b = blk[root[t]];          // the opener of a block carries its number
    key[t] = (uint64_t)(uint32_t)b << 32;
    id[t] = (int32_t)t;
}

__device__ __forceinline__ uint64_t fmix64(uint64_t x)
{  // 64-bit finaliser of MurmurHash3
    x ^= x >> 33; x *= 0xff51afd7ed558ccdULL;
    x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ULL;
    x ^= x >> 33;
    return x;
}

// segment list (items sorted by block, placement order inside a block), inverse tables, digest
__global__ void __launch_bounds__(256) kb_tables(PlanView pv, const uint64_t* __restrict__ blk_key, const int32_t* __restrict__ item,
                                                 const int2* __restrict__ rec, const int32_t* __restrict__ sorted_id,
                                                 int64_t n, int32_t L)
{
    __shared__ unsigned long long s_sum[8];
    if (pv.hdr->first_bad != kNoBad) return;
    const int64_t k = (int64_t)blockIdx.x * 256 + threadIdx.x;
    unsigned long long term = 0;
    if (k < n) {
        const int t = item[k];
        const int b = (int)(blk_key[k] >> 32);
        const int id = sorted_id[n - 1 - t];
        const int taken = rec[t].x;
        const int start = taken ? L - taken : 0;
        pv.seg_seq[k] = id;
        pv.seg_block[k] = b;
        pv.seg_start[k] = start;
        pv.seg_src[k] = pv.offsets[id];
        pv.seq_block[id] = b;
        pv.seq_start[id] = start;
        const uint64_t where = ((uint64_t)(uint32_t)b << 32) | (uint64_t)(uint32_t)start;
        term = fmix64(where * 0x9E3779B97F4A7C15ULL + (uint64_t)(uint32_t)id);
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) term += __shfl_xor_sync(kFull, term, d);
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) s_sum[w] = term;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) term += s_sum[i];
        atomicAdd(&pv.hdr->checksum, term);
    }
}

// per block: occupied slots (end of its last segment) and the widest block; block_seg_begin[b+1] was written by
// the bucket pass as "segments with block <= b"
__global__ void __launch_bounds__(256) kb_fills(PlanView pv, const int32_t* __restrict__ take_end, int64_t n)
{
    __shared__ int s_max[8];
    if (pv.hdr->first_bad != kNoBad) return;
    const int64_t n_blocks = take_end[0];          // items that opened a block
    const int64_t b = (int64_t)blockIdx.x * 256 + threadIdx.x;
    int segs = 0;
    if (b == 0) { pv.block_seg_begin[0] = 0; pv.hdr->n_blocks = n_blocks; }
    if (b < n_blocks) {
        const int k0 = b ? pv.block_seg_begin[b] : 0, k1 = pv.block_seg_begin[b + 1];
        const int last = k1 - 1;
        const int id = pv.seg_seq[last];
        pv.block_fill[b] = pv.seg_start[last] + (int)(pv.offsets[id + 1] - pv.offsets[id]);
        segs = k1 - k0;
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) segs = max(segs, __shfl_xor_sync(kFull, segs, d));
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) s_max[w] = segs;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) segs = max(segs, s_max[i]);
        atomicMax(&pv.hdr->max_segs, segs);
    }
}

__global__ void kb_finish(PlanHeader* h)
{
    if (threadIdx.x == 0 && blockIdx.x == 0 && h->first_bad == kNoBad) h->magic = kPlanMagic;
}

}  // namespace

size_t bfd_layout(int64_t n, int32_t t_block, void* base, BfdView* v)
{
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const size_t un = (size_t)n, ur = (size_t)t_block + 1;
    const size_t o_rec = take(sizeof(int2) * un), o_ka = take(8 * un), o_kb = take(8 * un), o_ia = take(4 * un),
                 o_ib = take(4 * un), o_put = take(4 * un), o_ja = take(4 * un), o_jb = take(4 * un), o_blk = take(4 * un),
                 o_pe = take(4 * ur), o_te = take(4 * ur);
    if (v) {
        char* b = static_cast<char*>(base);
        v->rec = reinterpret_cast<int2*>(b + o_rec);
        v->ek_a = reinterpret_cast<uint64_t*>(b + o_ka);
        v->ek_b = reinterpret_cast<uint64_t*>(b + o_kb);
        v->ei_a = reinterpret_cast<int32_t*>(b + o_ia);
        v->ei_b = reinterpret_cast<int32_t*>(b + o_ib);
        v->put_item = reinterpret_cast<int32_t*>(b + o_put);
        v->jump_a = reinterpret_cast<int32_t*>(b + o_ja);
        v->jump_b = reinterpret_cast<int32_t*>(b + o_jb);
        v->blk = reinterpret_cast<int32_t*>(b + o_blk);
        v->put_end = reinterpret_cast<int32_t*>(b + o_pe);
        v->take_end = reinterpret_cast<int32_t*>(b + o_te);
    }
    return off;
}

cudaError_t launch_bfd(const PlanView& pv, const WorkView& wv, const BfdView& bv, const uint64_t* sorted_key,
                       const int32_t* sorted_id, int64_t n, int32_t t_block, cudaStream_t st)
{
    const unsigned gn = (unsigned)((n + 255) / 256);
    const size_t smem = sizeof(int32_t) * (1024 + 64 + (size_t)t_block);
    cudaError_t e = opt_in_shared_memory(kb_chain, (int)smem);
    if (e != cudaSuccess) return e;
    kb_chain<<<1, 256, smem, st>>>(pv.hdr, sorted_key, bv.rec, (int32_t)n, t_block);
    int room_bits = 0;
    while ((1 << room_bits) <= t_block) ++room_bits;
    const int room_digits = (room_bits + 7) / 8;
    uint64_t* k_out;
    int32_t* i_out;
    // items ordered by (room they left, time)
    kb_event_keys<<<gn, 256, 0, st>>>(pv.hdr, bv.rec, n, bv.ek_a, bv.ei_a, 1);
    e = plan_radix_sort(bv.ek_a, bv.ei_a, bv.ek_b, bv.ei_b, n, 32, room_digits, wv.digit_hist, pv.hdr, st, &k_out, &i_out);
    if (e != cudaSuccess) return e;
    e = plan_key_buckets(k_out, n, t_block, bv.put_end, pv.hdr, st);
    if (e != cudaSuccess) return e;
    e = cudaMemcpyAsync(bv.put_item, i_out, sizeof(int32_t) * (size_t)n, cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return e;
    // items ordered by (room they took, time); room 0 = opened a block
    kb_event_keys<<<gn, 256, 0, st>>>(pv.hdr, bv.rec, n, bv.ek_a, bv.ei_a, 0);
    e = plan_radix_sort(bv.ek_a, bv.ei_a, bv.ek_b, bv.ei_b, n, 32, room_digits, wv.digit_hist, pv.hdr, st, &k_out, &i_out);
    if (e != cudaSuccess) return e;
    e = plan_key_buckets(k_out, n, t_block, bv.take_end, pv.hdr, st);
    if (e != cudaSuccess) return e;
    kb_pred<<<gn, 256, 0, st>>>(pv.hdr, k_out, i_out, bv.take_end, bv.put_item, bv.put_end, n, bv.jump_a, bv.blk);
    // pointer doubling: a block holds at most t_block items, so ceil(log2(t_block)) rounds reach every opener
    int32_t *jin = bv.jump_a, *jout = bv.jump_b;
    int rounds = 0;
    while ((1 << rounds) < t_block) ++rounds;
    for (int r = 0; r < rounds; ++r) {
        kb_jump<<<gn, 256, 0, st>>>(pv.hdr, jin, jout, n);
        int32_t* tmp = jin; jin = jout; jout = tmp;
    }
    // segments: items sorted by block (stable: placement order inside a block)
    kb_block_keys<<<gn, 256, 0, st>>>(pv.hdr, jin, bv.blk, n, bv.ek_a, bv.ei_a);
    int blk_bits = 0;
    while ((1LL << blk_bits) < n) ++blk_bits;
    const int blk_digits = blk_bits ? (blk_bits + 7) / 8 : 1;
    e = plan_radix_sort(bv.ek_a, bv.ei_a, bv.ek_b, bv.ei_b, n, 32, blk_digits, wv.digit_hist, pv.hdr, st, &k_out, &i_out);
    if (e != cudaSuccess) return e;
    e = plan_key_buckets(k_out, n, (int32_t)(n - 1), pv.block_seg_begin + 1, pv.hdr, st);
    if (e != cudaSuccess) return e;
    kb_tables<<<gn, 256, 0, st>>>(pv, k_out, i_out, bv.rec, sorted_id, n, t_block);
    kb_fills<<<gn, 256, 0, st>>>(pv, bv.take_end, n);
    kb_finish<<<1, 32, 0, st>>>(pv.hdr);
    count_launches(1 + 2 + 1 + rounds + 1 + 3);
    return cudaPeekAtLastError();
}

}  // namespace bload

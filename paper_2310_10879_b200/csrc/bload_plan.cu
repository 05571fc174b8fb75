// Planner kernels: ragged offsets, shuffle keys, key sort, the fill rule, inverse tables.
//
// The paper's block construction (Methods, first paragraph; caption of the pseudocode figure):
// open a block, draw a random unused sequence among those that still fit (Random_*() over L_dict),
// append it, repeat until nothing fits, pad, open the next block.  On the device this becomes
//   1. validate + exclusive scan of the lengths (ragged offsets), one Philox word per sequence
//      (shuffle key h_i) and one per draw (u_k);
//   2. a stable LSD radix sort of the ids by (T_i, h_i): L_dict as one array, buckets by length,
//      each bucket pre-shuffled;
//   3. the fill rule itself, a chain of n dependent draws run by one warp over a three-level table
//      of running counts kept in shared memory;
//   4. a parallel pass that resolves draws to sequence ids and writes the inverse tables.
#include <limits.h>

#include "bload_debug.cuh"
#include "bload_internal.cuh"

namespace bload {

namespace {

constexpr unsigned kFull = 0xffffffffu;
constexpr unsigned long long kNoBad = ULLONG_MAX;

// ---- Philox-4x64-10 (Salmon et al., SC'11): counter (idx,0,0,0), key (seed, stream); word 0 ----
__device__ __forceinline__ uint64_t philox_word0(uint64_t idx, uint64_t seed, uint64_t stream)
{
    const uint64_t M0 = 0xD2E7470EE14C6C93ULL, M1 = 0xCA5A826395121157ULL;
    const uint64_t W0 = 0x9E3779B97F4A7C15ULL, W1 = 0xBB67AE8584CAA73BULL;
    uint64_t c0 = idx, c1 = 0, c2 = 0, c3 = 0, k0 = seed, k1 = stream;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        if (r) { k0 += W0; k1 += W1; }
        uint64_t hi0 = __umul64hi(M0, c0), lo0 = M0 * c0;
        uint64_t hi1 = __umul64hi(M1, c2), lo1 = M1 * c2;
        c0 = hi1 ^ c1 ^ k0;
        c1 = lo1;
        c2 = hi0 ^ c3 ^ k1;
        c3 = lo0;
    }
    return c0;
}

// ---- block-wide exclusive scan over 256 threads (8 warps) ----
template <typename T>
__device__ __forceinline__ T warp_inclusive(T v)
{
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        T o = __shfl_up_sync(kFull, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

template <typename T, int WARPS>
__device__ __forceinline__ T block_exclusive(T v, T* warp_tot /*[WARPS] shared*/, T* total)
{
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    T inc = warp_inclusive(v);
    if (lane == 31) warp_tot[w] = inc;
    __syncthreads();
    T base = 0, tot = 0;
#pragma unroll
    for (int i = 0; i < WARPS; ++i) {
        T x = warp_tot[i];
        if (i < w) base += x;
        tot += x;
    }
    __syncthreads();
    *total = tot;
    return base + inc - v;
}

__global__ void k0_init(PlanHeader* h, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy)
{
    if (threadIdx.x == 0 && blockIdx.x == 0) {
        h->magic = 0;  // set when the plan is complete
        h->n = n;
        h->n_blocks = 0;
        h->sum_t = 0;
        h->first_bad = kNoBad;
        h->checksum = 0;
        h->seed = seed;
        h->t_block = t_block;
        h->t_max = 0;
        h->status = BLOAD_OK;
        h->max_segs = 0;
        h->policy = policy;
    }
}

// per-chunk sum of lengths, global max, first index with T outside [1, t_block]
__global__ void __launch_bounds__(256) k1_reduce(const int32_t* __restrict__ len, int64_t n, int32_t t_block,
                                                 int64_t* __restrict__ partial, PlanHeader* h)
{
    __shared__ int64_t s_sum[8];
    __shared__ int s_max[8];
    __shared__ unsigned long long s_bad[8];
    const int64_t base = (int64_t)blockIdx.x * kChunk;
    int64_t sum = 0;
    int mx = 0;
    unsigned long long bad = kNoBad;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int64_t i = base + e * 256 + threadIdx.x;
        if (i < n) {
            int t = len[i];
            if (t < 1 || t > t_block) { if ((unsigned long long)i < bad) bad = (unsigned long long)i; }
            sum += t;
            mx = max(mx, t);
        }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        sum += __shfl_xor_sync(kFull, sum, d);
        mx = max(mx, __shfl_xor_sync(kFull, mx, d));
        unsigned long long ob = __shfl_xor_sync(kFull, bad, d);
        bad = ob < bad ? ob : bad;
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { s_sum[w] = sum; s_max[w] = mx; s_bad[w] = bad; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) { sum += s_sum[i]; mx = max(mx, s_max[i]); bad = s_bad[i] < bad ? s_bad[i] : bad; }
        partial[blockIdx.x] = sum;
        atomicMax(&h->t_max, mx);
        if (bad != kNoBad) atomicMin(&h->first_bad, bad);
    }
}

// exclusive scan of the per-chunk sums (one CTA), total to the header, status on bad input
__global__ void __launch_bounds__(1024) k1_scan_partials(int64_t* __restrict__ partial, int64_t chunks, PlanHeader* h)
{
    __shared__ int64_t s_tot[32];
    int64_t carry = 0;
    for (int64_t lo = 0; lo < chunks; lo += 1024) {
        int64_t i = lo + threadIdx.x;
        int64_t v = i < chunks ? partial[i] : 0, tot;
        int64_t ex = block_exclusive<int64_t, 32>(v, s_tot, &tot);
        if (i < chunks) partial[i] = carry + ex;
        carry += tot;
    }
    if (threadIdx.x == 0) {
        h->sum_t = carry;
        if (h->first_bad != kNoBad) h->status = BLOAD_ERR_LENGTH;
    }
}

// offsets[i], sort key (T_i << 32 | h_i), payload id, random word of draw i
__global__ void __launch_bounds__(256) k1_offsets_keys(const int32_t* __restrict__ len, int64_t n, uint64_t seed,
                                                       const int64_t* __restrict__ partial,
                                                       int64_t* __restrict__ offsets, uint64_t* __restrict__ key,
                                                       int32_t* __restrict__ id, uint64_t* __restrict__ draw_u,
                                                       const PlanHeader* h)
{
    __shared__ int64_t s_tot[8];
    if (h->first_bad != kNoBad) return;
    const int64_t base = (int64_t)blockIdx.x * kChunk + (int64_t)threadIdx.x * 8;
    int t[8];
    int64_t sum = 0;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        t[e] = (base + e < n) ? len[base + e] : 0;
        sum += t[e];
    }
    int64_t tot;
    int64_t run = partial[blockIdx.x] + block_exclusive<int64_t, 8>(sum, s_tot, &tot);
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int64_t i = base + e;
        if (i < n) {
            offsets[i] = run;
            run += t[e];
            uint32_t hkey = (uint32_t)(philox_word0((uint64_t)i, seed, 1ULL) >> 32);
            key[i] = ((uint64_t)(uint32_t)t[e] << 32) | hkey;
            id[i] = (int32_t)i;
            draw_u[i] = philox_word0((uint64_t)i, seed, 2ULL);
            if (i == n - 1) offsets[n] = run;
        }
    }
}

// ---- stable LSD radix sort, 8-bit digits, chunk = 2048 keys per CTA ----
__global__ void __launch_bounds__(256) k3_hist(const uint64_t* __restrict__ key, int64_t n, int shift, int64_t chunks,
                                               uint32_t* __restrict__ hist, const PlanHeader* h)
{
    __shared__ uint32_t s_h[256];
    if (h->first_bad != kNoBad) return;
    s_h[threadIdx.x] = 0;
    __syncthreads();
    const int64_t base = (int64_t)blockIdx.x * kChunk;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int64_t i = base + e * 256 + threadIdx.x;
        if (i < n) atomicAdd(&s_h[(unsigned)(key[i] >> shift) & 255u], 1u);
    }
    __syncthreads();
    hist[(int64_t)threadIdx.x * chunks + blockIdx.x] = s_h[threadIdx.x];
}

// per digit: exclusive scan of its row of per-chunk counts (one warp per digit), row total to hist[256*chunks + d];
// the offsets of the digits themselves (a 256-entry scan of those totals) are formed by every scatter CTA
__global__ void __launch_bounds__(1024) k3_scan(uint32_t* __restrict__ hist, int64_t chunks, const PlanHeader* h)
{
    if (h->first_bad != kNoBad) return;
    const int lane = threadIdx.x & 31;
    const int d = (int)((blockIdx.x * blockDim.x + threadIdx.x) >> 5);  // 8 CTAs x 32 warps = 256 digits
    uint32_t* row = hist + (int64_t)d * chunks;
    uint32_t carry = 0;
    for (int64_t lo = 0; lo < chunks; lo += 32) {
        const int64_t i = lo + lane;
        const uint32_t v = i < chunks ? row[i] : 0;
        const uint32_t inc = warp_inclusive(v);
        if (i < chunks) row[i] = carry + inc - v;
        carry += __shfl_sync(kFull, inc, 31);
    }
    if (lane == 0) hist[256 * chunks + d] = carry;
}

__global__ void __launch_bounds__(256) k3_scatter(const uint64_t* __restrict__ key_in, const int32_t* __restrict__ id_in,
                                                  uint64_t* __restrict__ key_out, int32_t* __restrict__ id_out,
                                                  int64_t n, int shift, int64_t chunks,
                                                  const uint32_t* __restrict__ hist, const PlanHeader* h)
{
    __shared__ uint32_t s_cnt[8][256];
    __shared__ uint32_t s_tot[8];
    if (h->first_bad != kNoBad) return;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    for (int i = threadIdx.x; i < 8 * 256; i += 256) (&s_cnt[0][0])[i] = 0;
    __syncthreads();
    // warp w ranks its 256 consecutive keys, 32 at a time, in input order
    const int64_t wbase = (int64_t)blockIdx.x * kChunk + w * 256;
    uint64_t k[8];
    int32_t v[8];
    uint32_t rank[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int64_t i = wbase + e * 32 + lane;
        bool ok = i < n;
        k[e] = ok ? key_in[i] : 0;
        v[e] = ok ? id_in[i] : 0;
        unsigned d = (unsigned)(k[e] >> shift) & 255u;
        unsigned tag = ok ? d : (256u + lane);
        unsigned peers = __match_any_sync(kFull, tag);
        unsigned before = __popc(peers & ((1u << lane) - 1u));
        uint32_t prev = ok ? s_cnt[w][d] : 0;
        __syncwarp();
        if (ok && before == 0) s_cnt[w][d] = prev + __popc(peers);
        __syncwarp();
        rank[e] = prev + before;
    }
    __syncthreads();
    {
        const int d = threadIdx.x;
        uint32_t all;
        const uint32_t digit_base = block_exclusive<uint32_t, 8>(hist[256 * chunks + d], s_tot, &all);  // keys with a smaller digit
        uint32_t run = digit_base + hist[(int64_t)d * chunks + blockIdx.x];
#pragma unroll
        for (int ww = 0; ww < 8; ++ww) {
            uint32_t c = s_cnt[ww][d];
            s_cnt[ww][d] = run;
            run += c;
        }
    }
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        int64_t i = wbase + e * 32 + lane;
        if (i < n) {
            unsigned d = (unsigned)(k[e] >> shift) & 255u;
            uint32_t p = s_cnt[w][d] + rank[e];
            key_out[p] = k[e];
            id_out[p] = v[e];
        }
    }
}

// bucket_end[l] = number of sequences with length <= l, l = 0..t_block, from the sorted keys
__global__ void __launch_bounds__(256) k3_buckets(const uint64_t* __restrict__ key, int64_t n, int32_t t_block,
                                                  int32_t* __restrict__ bucket_end, const PlanHeader* h)
{
    if (h->first_bad != kNoBad) return;
    int64_t p = (int64_t)blockIdx.x * 256 + threadIdx.x;
    if (p >= n) return;
    int t = (int)(key[p] >> 32);
    if (p == 0)
        for (int l = 0; l < t; ++l) bucket_end[l] = 0;
    int tn = (p + 1 < n) ? (int)(key[p + 1] >> 32) : t_block + 1;
    for (int l = t; l < tn; ++l) bucket_end[l] = (int32_t)(p + 1);
}

// ---- the fill rule: one warp, n dependent draws ----
// Shared memory holds running counts of UNUSED sequences as a three-level, 32-ary table of prefix sums
// over the lengths (leaf x stands for length x + 1; x = a*1024 + b*32 + c).  Every row has 33 entries:
// entry 0 is zero and entry i+1 is the inclusive sum up to digit i, so that the same row serves as
// inclusive prefix (read at digit+1) and exclusive prefix (read at digit) without a select or a shuffle,
// and rows of 33 words fall on distinct banks:
//   Q0[a+1]            sequences with x < (a+1)*1024
//   Q1[a][b+1]         sequences with a*1024 <= x < a*1024 + (b+1)*32
//   Q2[a*32+b][c+1]    sequences with (a*32+b)*32 <= x <= (a*32+b)*32 + c
// "How many fit in r slots" is three reads; "the j-th of them in order of length" is one
// compare + ballot + popcount per level with one entry per lane; a draw then decrements the entries
// at and after the chosen digit in one row per level.
constexpr int kQ1Off = 36, kRingOff = kQ1Off + 32 * 33, kQ2Off = kRingOff + 128;  // in 32-bit words; ring 16-byte aligned
static_assert(kRingOff % 4 == 0, "ring alignment");

//
// RESUME: the chain runs in several launches ("chunks") so that blocks which are already closed can be packed on
// another stream while later ones are still being built.  A chunk stops at the first block that closes at or after
// draw `k_target`, leaves its position in `rs` and its count tables in `snap`, and records the blocks and draws it
// covered; the next launch picks both up.  Without RESUME the kernel is the single launch it always was.
template <bool RESUME>
__global__ void __launch_bounds__(256, 1) k4_fill(PlanView pv, const int32_t* __restrict__ bucket_end,
                                                  const uint64_t* __restrict__ draw_u, int4* __restrict__ draw_rec,
                                                  int64_t n64, int32_t L, FillResume* __restrict__ rs,
                                                  int32_t* __restrict__ snap, int32_t k_target, int32_t filler_end)
{
    extern __shared__ __align__(16) int32_t sm[];
    int32_t* Q0 = sm;                                      // [33]
    int32_t* Q1 = sm + kQ1Off;                             // [32][33]
    int4* ring = reinterpret_cast<int4*>(sm + kRingOff);   // [32] records of the last draws
    int32_t* Q2 = sm + kQ2Off;                             // [rows][33], rows = ceil(L / 32)
    if (pv.hdr->first_bad != kNoBad) return;
    const int rows = (L + 31) >> 5;
    const int chunk = RESUME ? rs->chunk : 0;
    if (RESUME && rs->done) {  // an earlier chunk placed the last sequence: this one covers nothing
        __syncthreads();       // every thread has read the state before thread 0 changes it
        if (threadIdx.x == 0) {
            const int e = rs->range[chunk - 1][1], d = rs->draw[chunk - 1][1], eb = rs->draw[chunk - 1][3];
            rs->range[chunk][0] = e; rs->range[chunk][1] = e; rs->range[chunk][2] = e;
            rs->draw[chunk][0] = d; rs->draw[chunk][1] = d; rs->draw[chunk][2] = eb; rs->draw[chunk][3] = eb;
            rs->chunk = chunk + 1;
        }
        return;
    }
    if (RESUME && chunk > 0) {
        const int words = kQ2Off + rows * 33;
        for (int i = threadIdx.x; i < words; i += blockDim.x) sm[i] = snap[i];
    } else {
        auto upto = [&](int l) { return bucket_end[min(l, L)]; };  // sequences with length <= l
        for (int idx = threadIdx.x; idx < rows * 32; idx += blockDim.x)
            Q2[(idx >> 5) * 33 + (idx & 31) + 1] = upto(idx + 1) - upto(idx & ~31);
        for (int r = threadIdx.x; r < rows; r += blockDim.x) Q2[r * 33] = 0;
        for (int idx = threadIdx.x; idx < 1024; idx += blockDim.x)
            Q1[(idx >> 5) * 33 + (idx & 31) + 1] = upto((idx + 1) << 5) - upto((idx >> 5) << 10);
        if (threadIdx.x < 32) { Q1[threadIdx.x * 33] = 0; Q0[threadIdx.x + 1] = upto((threadIdx.x + 1) << 10); }
        if (threadIdx.x == 0) Q0[0] = 0;
    }
    int k = 0, b = 0, room = L, start = 0;
    if (RESUME && chunk > 0) { k = rs->k; b = rs->b; room = rs->room; start = rs->start; }
    __syncthreads();
    if (threadIdx.x >= 32) return;

    const int lane = threadIdx.x;
    const int n = (int)n64;
    int q0 = Q0[lane + 1];
    int f0 = Q0[1];         // unused sequences of length <= 1024 (every lane keeps a copy)
    int r1 = Q1[lane + 1];  // row 0 of level 1, this lane's entry (the shared-memory copy stays current for the m lookup)
    const int k_first = k, b_first = b;
    int flush_from = k & 31;  // records of the first group below this lane were written by the previous chunk
    if (lane == 0 && k == 0) pv.block_seg_begin[0] = 0;
    // random words of 32 draws at a time, one per lane, the next 32 prefetched
    uint64_t u_cur = (k & ~31) + lane < n ? draw_u[(k & ~31) + lane] : 0;
    uint64_t u_nxt = (k & ~31) + 32 + lane < n ? draw_u[(k & ~31) + 32 + lane] : 0;
    // m = unused sequences that fit into the room left.  A block is only ever (re)opened here with room == L, where
    // every unused sequence fits; inside a block the next m comes out of the previous draw (see below).
    int m = n - k;
    // One draw; `slot` = k & 31, the draw's place in its group of 32 (ring entry, lane that holds its random word).
    // Returns true when the chain has to stop here (RESUME only: a block closed at or after the chunk's target).
    auto draw = [&](const int slot) -> bool {
        if (m == 0) {  // nothing fits: the rest of the block is padding
            if (lane == 0) { pv.block_fill[b] = start; pv.block_seg_begin[b + 1] = k; }
            ++b; room = L; start = 0;
            m = n - k;
            if (RESUME && k >= k_target) return true;
        }
        const uint64_t u = __shfl_sync(kFull, u_cur, slot);
        // j = floor(u * m / 2^64), m < 2^31, from 32-bit pieces
        int j = (int)(((uint64_t)(uint32_t)(u >> 32) * (uint32_t)m + __umulhi((uint32_t)u, (uint32_t)m)) >> 32);
        // level 0 -- skipped when the pick lies among the lengths 1..1024, whose level-1 row is kept in registers:
        // that takes a vote and a dependent shared-memory load off the chain for most draws (measured 202 -> 177 ns
        // per draw on heavy-tailed lengths, 215 -> 200 ns on token lengths).  Inside the branch a >= 1, because
        // lane 0 holds q0 == f0 <= j.
        int a = 0, q1 = r1;
        if (j >= f0) {
            a = __popc(__ballot_sync(kFull, q0 <= j));
            j -= Q0[a];
            q1 = Q1[a * 33 + lane + 1];
        }
        // level 1
        const int bb = __popc(__ballot_sync(kFull, q1 <= j));
        const int row = (a << 5) + bb;
        const int q2 = Q2[row * 33 + lane + 1];
        const int below = Q2[row * 33 + lane];
        j -= Q1[a * 33 + bb];
        // While the level-2 vote is under way every lane looks up how many sequences would fit after ITS candidate
        // length row*32 + lane + 1 (tables as they are before this draw, minus the drawn sequence itself when it
        // would still fit); the chosen lane's value is the next draw's m.  That keeps the three-load lookup off the
        // chain (177 -> 162 ns per draw).  The slot is clamped to >= 0, and is < L, so the indices stay in the tables.
        const int my_len = (row << 5) + lane + 1;
        const int my_room = room - my_len;
        const int yy = max(my_room - 1, 0), yya = yy >> 10, yyr = yy >> 5;
        int my_m = Q2[yyr * 33 + (yy & 31) + 1] + Q1[yya * 33 + (yyr & 31)] + Q0[yya];
        my_m = my_room > 0 ? my_m - (my_len <= my_room ? 1 : 0) : 0;
        // level 2
        const int c = __popc(__ballot_sync(kFull, q2 <= j));
        const int len = (row << 5) + c + 1;
        m = __shfl_sync(kFull, my_m, c);
        // decrement the running counts at and after the chosen digits
        if (lane >= a) { --q0; Q0[lane + 1] = q0; }
        if (a == 0) { --f0; if (lane >= bb) r1 = q1 - 1; }
        if (lane >= bb) Q1[a * 33 + lane + 1] = q1 - 1;
        if (lane >= c) Q2[row * 33 + lane + 1] = q2 - 1;
        // the draw's record goes to a 32-entry ring in shared memory and leaves 32 at a time, one per lane:
        // a global store inside the chain costs about 55 cycles per draw
        if (lane == c) ring[slot] = make_int4(len, q2 - below, b, start);  // q2 - below: unused of this length
        room -= len; start += len; ++k;
        return false;
    };
    // a full group of 32 records leaves the ring, and the random words of the next group move up
    auto flush_group = [&]() {
        __syncwarp();
        if (!RESUME || lane >= flush_from) draw_rec[k - 32 + lane] = ring[lane];
        flush_from = 0;
        u_cur = u_nxt;
        u_nxt = k + 32 + lane < n ? draw_u[k + 32 + lane] : 0;
        __syncwarp();
    };
    // The loop is unrolled over half a group: ring entry and word lane become a base plus a constant, and the flush
    // test and the loop branch come once per 16 draws.  Measured per draw, heavy-tailed / token lengths: rolled loop
    // 162 / 184 ns, unrolled 4 times 153 / 166, 8 times 148 / 162, 16 times 147 / 160, 32 times 142 / 155 -- but the
    // last figure moved between 142 and 159 ns from one build or process to the next (the body of 32 draws no longer
    // fits the innermost instruction cache), while 8 and 16 repeated to the tenth of a nanosecond.  Draws before the
    // first boundary (a resumed chain) and after the last whole half group go one by one.
    constexpr int kUnroll = 16;
    bool stop = false;
    while (!stop && k < n && (k & (kUnroll - 1)) != 0) {
        stop = draw(k & 31);
        if (!stop && (k & 31) == 0) flush_group();
    }
    while (!stop && k + kUnroll <= n) {
        const int base = k & 31;
#pragma unroll
        for (int i = 0; i < kUnroll; ++i) {
            if (draw(base + i)) { stop = true; break; }
        }
        if (!stop && (k & 31) == 0) flush_group();
    }
    while (!stop && k < n) {
        stop = draw(k & 31);
        if (!stop && (k & 31) == 0) flush_group();
    }
    __syncwarp();
    if (lane < (k & 31) && lane >= flush_from) draw_rec[(k & ~31) + lane] = ring[lane];
    const bool finished = k == n;
    if (finished && lane == 0) {
        pv.block_fill[b] = start;
        pv.block_seg_begin[b + 1] = k;
        pv.hdr->n_blocks = b + 1;
    }
    if (RESUME) {
        const int closed = finished ? b + 1 : b;  // blocks [b_first, closed) are complete now
        __syncwarp();
        const int words = kQ2Off + rows * 33;
        if (!finished)
            for (int i = lane; i < words; i += 32) snap[i] = sm[i];
        if (lane == 0) {
            rs->k = k; rs->b = b; rs->room = room; rs->start = start;
            rs->done = finished ? 1 : 0;
            // what the copies may touch is clamped to the rows the caller's buffers have (filler_end)
            const int lo_c = min(b_first, filler_end), hi_c = min(closed, filler_end);
            rs->range[chunk][0] = lo_c; rs->range[chunk][1] = hi_c; rs->range[chunk][2] = hi_c;
            rs->draw[chunk][0] = k_first; rs->draw[chunk][1] = k; rs->draw[chunk][2] = b_first; rs->draw[chunk][3] = closed;
            rs->chunk = chunk + 1;
            if (finished) {  // the filler blocks between the end of the plan and the end of the caller's buffers
                rs->range[kMaxEpochChunks][0] = hi_c;
                rs->range[kMaxEpochChunks][1] = filler_end;
                rs->range[kMaxEpochChunks][2] = hi_c;
            }
        }
    }
}

// Policy 1: every LENGTH that fits and still has an unused sequence is equally likely (the other reading
// of "a random entry of L_dict": a random key of the dictionary).  Same three-level table, but it counts
// non-exhausted lengths instead of sequences, and a leaf word packs two fields:
//   bits 0..5   inclusive count of non-exhausted lengths in its row up to this leaf (0..32)
//   bits 6..31  unused sequences of this length (hence n < 2^26 for this policy)
// Most draws change only the chosen leaf's count; the prefix fields move when a length runs out.
__global__ void __launch_bounds__(256, 1) k4_fill_lengths(PlanView pv, const int32_t* __restrict__ bucket_end,
                                                          const uint64_t* __restrict__ draw_u,
                                                          int4* __restrict__ draw_rec, int64_t n64, int32_t L)
{
    extern __shared__ __align__(16) int32_t sm[];
    int32_t* Q0 = sm;                                      // [33], entry 0 is zero (see k4_fill)
    int32_t* Q1 = sm + kQ1Off;                             // [32][33]
    int4* ring = reinterpret_cast<int4*>(sm + kRingOff);
    int32_t* Q2 = sm + kQ2Off;                             // [rows][32] packed leaf words (rows are not shifted)
    if (pv.hdr->first_bad != kNoBad) return;
    const int rows = (L + 31) >> 5;
    auto upto = [&](int l) { return bucket_end[min(l, L)]; };
    // leaves: one thread per row, 32 leaves in order
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        int live = 0;
        for (int c = 0; c < 32; ++c) {
            const int x = (r << 5) + c;
            const int cnt = x < L ? upto(x + 1) - upto(x) : 0;
            live += cnt > 0;
            Q2[x] = (int32_t)(((uint32_t)cnt << 6) | (uint32_t)live);
        }
    }
    __syncthreads();
    // rows of a top group: one thread per group
    if (threadIdx.x < 32) {
        int run = 0;
        for (int b = 0; b < 32; ++b) {
            const int r = (threadIdx.x << 5) + b;
            run += r < rows ? (Q2[(r << 5) + 31] & 63) : 0;
            Q1[threadIdx.x * 33 + b + 1] = run;
        }
        Q1[threadIdx.x * 33] = 0;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        int run = 0;
        Q0[0] = 0;
        for (int a = 0; a < 32; ++a) { run += Q1[a * 33 + 32]; Q0[a + 1] = run; }
    }
    __syncthreads();
    if (threadIdx.x >= 32) return;

    const int lane = threadIdx.x;
    const int n = (int)n64;
    int q0 = Q0[lane + 1];
    int f0 = Q0[1];         // live lengths <= 1024 (every lane keeps a copy)
    int r1 = Q1[lane + 1];  // row 0 of level 1 in registers, as in k4_fill
    int live = Q0[32];      // lengths that still have an unused sequence
    int k = 0, b = 0, room = L, start = 0;
    if (lane == 0) pv.block_seg_begin[0] = 0;
    uint64_t u_cur = lane < n ? draw_u[lane] : 0;
    uint64_t u_nxt = 32 + lane < n ? draw_u[32 + lane] : 0;
    // m = lengths that fit and are not exhausted; every live length fits into a freshly opened block, and inside a
    // block the next m comes out of the previous draw (per candidate lane, as in k4_fill)
    int m = live;
    // one draw; `slot` = k & 31 (ring entry, lane of the random word): see k4_fill
    auto draw = [&](const int slot) {
        if (m == 0) {
            if (lane == 0) { pv.block_fill[b] = start; pv.block_seg_begin[b + 1] = k; }
            ++b; room = L; start = 0;
            m = live;
        }
        const uint64_t u = __shfl_sync(kFull, u_cur, slot);
        int j = (int)(((uint64_t)(uint32_t)(u >> 32) * (uint32_t)m + __umulhi((uint32_t)u, (uint32_t)m)) >> 32);
        int a = 0, q1 = r1;
        if (j >= f0) {  // beyond the lengths <= 1024: walk level 0 (a >= 1 here, lane 0 holds q0 == f0 <= j)
            a = __popc(__ballot_sync(kFull, q0 <= j));
            j -= Q0[a];
            q1 = Q1[a * 33 + lane + 1];
        }
        const int bb = __popc(__ballot_sync(kFull, q1 <= j));
        const int row = (a << 5) + bb;
        const int q2 = Q2[(row << 5) + lane];
        j -= Q1[a * 33 + bb];
        // the next m for this lane's candidate length (old tables; the length itself leaves the count when this draw
        // takes its last sequence and it would still fit); slot clamped to [0, L)
        const int my_len = (row << 5) + lane + 1;
        const int my_room = room - my_len;
        const int yy = max(my_room - 1, 0), yya = yy >> 10;
        int my_m = (Q2[yy] & 63) + Q1[yya * 33 + ((yy >> 5) & 31)] + Q0[yya];
        my_m = my_room > 0 ? my_m - ((((uint32_t)q2 >> 6) == 1u && my_len <= my_room) ? 1 : 0) : 0;
        const int c = __popc(__ballot_sync(kFull, (q2 & 63) <= j));
        const int len = (row << 5) + c + 1;
        const int cnt = (int)((uint32_t)__shfl_sync(kFull, q2, c) >> 6);  // unused sequences of the chosen length, >= 1
        m = __shfl_sync(kFull, my_m, c);
        if (cnt == 1) {  // the length runs out: it leaves the prefix counts of all three levels
            --live;
            if (lane >= a) { --q0; Q0[lane + 1] = q0; }
            if (a == 0) { --f0; if (lane >= bb) r1 = q1 - 1; }
            if (lane >= bb) Q1[a * 33 + lane + 1] = q1 - 1;
            if (lane >= c) Q2[(row << 5) + lane] = (lane == c ? q2 - 64 : q2) - 1;
        } else if (lane == c) {
            Q2[(row << 5) + lane] = q2 - 64;
        }
        if (lane == c) ring[slot] = make_int4(len, cnt, b, start);
        room -= len; start += len; ++k;
    };
    auto flush_group = [&]() {
        __syncwarp();
        draw_rec[k - 32 + lane] = ring[lane];
        u_cur = u_nxt;
        u_nxt = k + 32 + lane < n ? draw_u[k + 32 + lane] : 0;
        __syncwarp();
    };
    while (k + 16 <= n) {  // unrolled over half a group, as in k4_fill
        const int base = k & 31;
#pragma unroll
        for (int i = 0; i < 16; ++i) draw(base + i);
        if ((k & 31) == 0) flush_group();
    }
    while (k < n) {
        draw(k & 31);
        if ((k & 31) == 0) flush_group();
    }
    __syncwarp();
    if (lane < (n & 31)) draw_rec[(n & ~31) + lane] = ring[lane];
    if (lane == 0) {
        pv.block_fill[b] = start;
        pv.block_seg_begin[b + 1] = k;
        pv.hdr->n_blocks = b + 1;
    }
}

__device__ __forceinline__ uint64_t fmix64(uint64_t x)
{  // 64-bit finaliser of MurmurHash3
    x ^= x >> 33; x *= 0xff51afd7ed558ccdULL;
    x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ULL;
    x ^= x >> 33;
    return x;
}

// resolve draws to sequence ids; segment list, inverse tables, digest, widest block.  With `draw_range` the kernel
// covers the draws [draw_range[0], draw_range[1]) and the blocks [draw_range[2], draw_range[3]) of one chunk of
// a plan that is still being built (every block has at least one draw, so the draw index doubles as block index).
__global__ void __launch_bounds__(256) k5_tables(PlanView pv, const int4* __restrict__ draw_rec,
                                                 const int32_t* __restrict__ bucket_end,
                                                 const int32_t* __restrict__ sorted_id, int64_t n,
                                                 const int32_t* __restrict__ draw_range)
{
    __shared__ unsigned long long s_sum[8];
    __shared__ int s_max[8];
    if (pv.hdr->first_bad != kNoBad) return;
    const int64_t k_lo = draw_range ? draw_range[0] : 0, k_hi = draw_range ? draw_range[1] : n;
    const int64_t b_lo = draw_range ? draw_range[2] : 0;
    const int64_t b_hi = draw_range ? draw_range[3] : pv.hdr->n_blocks;
    unsigned long long term = 0;
    int segs = 0;
    for (int64_t k = k_lo + (int64_t)blockIdx.x * 256 + threadIdx.x; k < k_hi; k += (int64_t)gridDim.x * 256) {
        if (!BLOAD_MAY_READ(draw_rec + k, 16)) continue;
        int4 r = draw_rec[k];
        if (!BLOAD_MAY_READ(bucket_end + r.x, 4) || !BLOAD_MAY_READ(sorted_id + (bucket_end[r.x] - r.y), 4)) continue;
        int id = sorted_id[bucket_end[r.x] - r.y];
        if (!(BLOAD_MAY_WRITE(pv.seg_seq + k, 4) && BLOAD_MAY_WRITE(pv.seg_block + k, 4) && BLOAD_MAY_WRITE(pv.seg_start + k, 4) &&
              BLOAD_MAY_WRITE(pv.seg_src + k, 8) && BLOAD_MAY_READ(pv.offsets + id, 8) && BLOAD_MAY_WRITE(pv.seq_block + id, 4) &&
              BLOAD_MAY_WRITE(pv.seq_start + id, 4)))
            continue;
        pv.seg_seq[k] = id;
        pv.seg_block[k] = r.z;
        pv.seg_start[k] = r.w;
        pv.seg_src[k] = pv.offsets[id];
        pv.seq_block[id] = r.z;
        pv.seq_start[id] = r.w;
        uint64_t where = ((uint64_t)(uint32_t)r.z << 32) | (uint64_t)(uint32_t)r.w;
        term += fmix64(where * 0x9E3779B97F4A7C15ULL + (uint64_t)(uint32_t)id);
        const int64_t b = b_lo + (k - k_lo);
        if (b < b_hi) segs = max(segs, pv.block_seg_begin[b + 1] - pv.block_seg_begin[b]);
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) {
        term += __shfl_xor_sync(kFull, term, d);
        segs = max(segs, __shfl_xor_sync(kFull, segs, d));
    }
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (lane == 0) { s_sum[w] = term; s_max[w] = segs; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int i = 1; i < 8; ++i) { term += s_sum[i]; segs = max(segs, s_max[i]); }
        if (term) atomicAdd(&pv.hdr->checksum, term);
        if (segs) atomicMax(&pv.hdr->max_segs, segs);
    }
}

__global__ void k5_finish(PlanHeader* h)
{
    if (threadIdx.x == 0 && blockIdx.x == 0 && h->first_bad == kNoBad) h->magic = kPlanMagic;
}

}  // namespace

size_t work_layout(int64_t n, int32_t t_block, void* base, WorkView* w)
{
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const int64_t chunks = chunks_of(n);
    size_t o_ka = take(sizeof(uint64_t) * n), o_kb = take(sizeof(uint64_t) * n);
    size_t o_ia = take(sizeof(int32_t) * n), o_ib = take(sizeof(int32_t) * n);
    size_t o_u = take(sizeof(uint64_t) * n), o_rec = take(sizeof(int4) * n);
    size_t o_part = take(sizeof(int64_t) * chunks), o_hist = take(sizeof(uint32_t) * 256 * (chunks + 1));
    size_t o_be = take(sizeof(int32_t) * ((size_t)t_block + 1));
    if (w) {
        char* b = static_cast<char*>(base);
        w->key_a = reinterpret_cast<uint64_t*>(b + o_ka);
        w->key_b = reinterpret_cast<uint64_t*>(b + o_kb);
        w->id_a = reinterpret_cast<int32_t*>(b + o_ia);
        w->id_b = reinterpret_cast<int32_t*>(b + o_ib);
        w->draw_u = reinterpret_cast<uint64_t*>(b + o_u);
        w->draw_rec = reinterpret_cast<int4*>(b + o_rec);
        w->partial = reinterpret_cast<int64_t*>(b + o_part);
        w->digit_hist = reinterpret_cast<uint32_t*>(b + o_hist);
        w->bucket_end = reinterpret_cast<int32_t*>(b + o_be);
    }
    return off;
}

cudaError_t plan_radix_sort(uint64_t* ka, int32_t* ia, uint64_t* kb, int32_t* ib, int64_t n, int first_shift, int digits,
                            uint32_t* hist, const PlanHeader* hdr, cudaStream_t st, uint64_t** k_out, int32_t** i_out)
{
    const int64_t chunks = chunks_of(n);
    const unsigned gc = (unsigned)chunks;
    uint64_t *kin = ka, *kout = kb;
    int32_t *iin = ia, *iout = ib;
    for (int p = 0; p < digits; ++p) {
        const int shift = first_shift + 8 * p;
        k3_hist<<<gc, 256, 0, st>>>(kin, n, shift, chunks, hist, hdr);
        k3_scan<<<8, 1024, 0, st>>>(hist, chunks, hdr);
        k3_scatter<<<gc, 256, 0, st>>>(kin, iin, kout, iout, n, shift, chunks, hist, hdr);
        uint64_t* tk = kin; kin = kout; kout = tk;
        int32_t* ti = iin; iin = iout; iout = ti;
    }
    count_launches(3 * digits);
    *k_out = kin; *i_out = iin;
    return cudaPeekAtLastError();
}

cudaError_t plan_key_buckets(const uint64_t* sorted_keys, int64_t n, int32_t max_value, int32_t* bucket_end,
                             const PlanHeader* hdr, cudaStream_t st)
{
    k3_buckets<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(sorted_keys, n, max_value, bucket_end, hdr);
    count_launches(1);
    return cudaPeekAtLastError();
}

size_t epoch_layout(int32_t t_block, void* base, EpochView* v)
{
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const size_t o_rs = take(sizeof(FillResume));
    const size_t o_tab = take(sizeof(int32_t) * (kQ2Off + (size_t)((t_block + 31) / 32) * 33));
    if (v) {
        char* b = static_cast<char*>(base);
        v->resume = reinterpret_cast<FillResume*>(b + o_rs);
        v->fill_tables = reinterpret_cast<int32_t*>(b + o_tab);
    }
    return off;
}

// validate + scan + keys + key sort + buckets; *sorted_id receives the array of ids sorted by (T, h)
cudaError_t launch_plan_front(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                              const PlanView& pv, const WorkView& wv, cudaStream_t st, int32_t** sorted_id,
                              uint64_t** sorted_key, cudaEvent_t* ev)
{
    const int64_t chunks = chunks_of(n);
    const unsigned gc = (unsigned)chunks;
    if (ev) cudaEventRecord(ev[0], st);
    k0_init<<<1, 32, 0, st>>>(pv.hdr, n, t_block, seed, policy);
    k1_reduce<<<gc, 256, 0, st>>>(d_lengths, n, t_block, wv.partial, pv.hdr);
    k1_scan_partials<<<1, 1024, 0, st>>>(wv.partial, chunks, pv.hdr);
    k1_offsets_keys<<<gc, 256, 0, st>>>(d_lengths, n, seed, wv.partial, pv.offsets, wv.key_a, wv.id_a, wv.draw_u, pv.hdr);
    if (ev) cudaEventRecord(ev[1], st);

    // digits: 4 of the shuffle key, then as many as the block length needs
    int t_bits = 0;
    while ((1 << t_bits) <= t_block) ++t_bits;
    const int passes = 4 + (t_bits + 7) / 8;
    uint64_t *kin = wv.key_a, *kout = wv.key_b;
    int32_t *iin = wv.id_a, *iout = wv.id_b;
    for (int p = 0; p < passes; ++p) {
        const int shift = 8 * p;
        k3_hist<<<gc, 256, 0, st>>>(kin, n, shift, chunks, wv.digit_hist, pv.hdr);
        k3_scan<<<8, 1024, 0, st>>>(wv.digit_hist, chunks, pv.hdr);
        k3_scatter<<<gc, 256, 0, st>>>(kin, iin, kout, iout, n, shift, chunks, wv.digit_hist, pv.hdr);
        uint64_t* tk = kin; kin = kout; kout = tk;
        int32_t* ti = iin; iin = iout; iout = ti;
    }
    k3_buckets<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(kin, n, t_block, wv.bucket_end, pv.hdr);
    if (ev) cudaEventRecord(ev[2], st);
    count_launches(4 + 3 * passes + 1);
    *sorted_id = iin;
    if (sorted_key) *sorted_key = kin;
    return cudaPeekAtLastError();
}

cudaError_t launch_plan_front(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                              const PlanView& pv, const WorkView& wv, cudaStream_t st, int32_t** sorted_id)
{
    return launch_plan_front(d_lengths, n, t_block, seed, policy, pv, wv, st, sorted_id, nullptr, nullptr);
}

static size_t fill_smem_bytes(int32_t t_block) { return sizeof(int32_t) * (kQ2Off + (size_t)((t_block + 31) / 32) * 33); }

cudaError_t launch_fill_chunk(const PlanView& pv, const WorkView& wv, const EpochView& ev, int64_t n, int32_t t_block,
                              int32_t k_target, int32_t filler_end, cudaStream_t st)
{
    size_t smem = fill_smem_bytes(t_block);
    if (smem < (size_t)kChainSmemBytes) smem = kChainSmemBytes;  // keeps other CTAs off this SM (see kChainSmemBytes)
    cudaError_t e = opt_in_shared_memory(k4_fill<true>, (int)smem);
    if (e != cudaSuccess) return e;
    k4_fill<true><<<1, 256, smem, st>>>(pv, wv.bucket_end, wv.draw_u, wv.draw_rec, n, t_block, ev.resume, ev.fill_tables,
                                         k_target, filler_end);
    count_launches(1);
    return cudaPeekAtLastError();
}

cudaError_t launch_tables_chunk(const PlanView& pv, const WorkView& wv, const int32_t* sorted_id, int64_t n,
                                const int32_t* d_draw_range, cudaStream_t st)
{
    const int64_t want = (n + 255) / 256, cap = (int64_t)device_info().sm_count * 4;
    BLOAD_DBG_UNCHECKED(st);  // runs beside launches of another stream
    k5_tables<<<(unsigned)(want < cap ? want : cap), 256, kBesideChainSmemBytes, st>>>(pv, wv.draw_rec, wv.bucket_end, sorted_id, n,
                                                                                        d_draw_range);
    count_launches(1);
    return cudaPeekAtLastError();
}

cudaError_t launch_plan_finish(const PlanView& pv, cudaStream_t st)
{
    k5_finish<<<1, 32, 0, st>>>(pv.hdr);
    count_launches(1);
    return cudaPeekAtLastError();
}

cudaError_t launch_plan(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                        const PlanView& pv, const WorkView& wv, cudaStream_t st, cudaEvent_t* ev, const BfdView* bv)
{
    int32_t* iin = nullptr;
    uint64_t* kin = nullptr;
    cudaError_t e = launch_plan_front(d_lengths, n, t_block, seed, policy, pv, wv, st, &iin, &kin, ev);
    if (e != cudaSuccess) return e;
    if (policy == BLOAD_POLICY_BEST_FIT_DECREASING) {  // a different planner from here on (see bload_bfd.cu)
        cudaError_t eb = bv ? launch_bfd(pv, wv, *bv, kin, iin, n, t_block, st) : cudaErrorInvalidValue;
        if (ev) { cudaEventRecord(ev[3], st); cudaEventRecord(ev[4], st); }
        return eb;
    }
    const size_t smem = fill_smem_bytes(t_block);
    if (policy == BLOAD_POLICY_UNIFORM_LENGTHS) {
        e = opt_in_shared_memory(k4_fill_lengths, (int)smem);
        if (e != cudaSuccess) return e;
        k4_fill_lengths<<<1, 256, smem, st>>>(pv, wv.bucket_end, wv.draw_u, wv.draw_rec, n, t_block);
    } else {
        e = opt_in_shared_memory(k4_fill<false>, (int)smem);
        if (e != cudaSuccess) return e;
        k4_fill<false><<<1, 256, smem, st>>>(pv, wv.bucket_end, wv.draw_u, wv.draw_rec, n, t_block, nullptr, nullptr, 0, 0);
    }
    if (ev) cudaEventRecord(ev[3], st);

    {   // the table kernel may touch the plan buffer and the scratch buffer, nothing else
        bload_sizes_t sz;
        plan_layout(n, &sz);
        const size_t work_bytes = work_layout(n, t_block, nullptr, nullptr);
        BLOAD_DBG_EXPECT(st, dbg::kTables, {{pv.hdr, sz.plan_bytes}, {wv.key_a, work_bytes}}, {{pv.hdr, sz.plan_bytes}});
    }
    k5_tables<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(pv, wv.draw_rec, wv.bucket_end, iin, n, nullptr);
    k5_finish<<<1, 32, 0, st>>>(pv.hdr);
    count_launches(1 + 2);
    if (ev) cudaEventRecord(ev[4], st);
    return cudaPeekAtLastError();
}

}  // namespace bload

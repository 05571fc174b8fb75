// The chunking strategy the paper compares with (section "Problem Statement and Current Limitations": each sample
// is broken into chunks of T_block frames and each chunk is treated as an individual sample; figure "Sampling
// solution"; Table I, column "sampling").  It is a planner only: it writes ordinary plan tables in which chunk j is
// "sequence" j and fills block j from slot 0, so that the pack, unpack, metadata and consumer kernels run unchanged.
//   kc_scan    one CTA walks the sequences with a running carry: first frame and first chunk number of every
//              sequence, and the totals (chunks, frames kept / deleted, padding, longest sequence, first bad length);
//   kc_tables  one thread per chunk: finds its sequence by binary search of the chunk numbers and writes its row of
//              every table; the plan's digest is summed per warp.
#include <string.h>

#include "bload_internal.cuh"

namespace bload {

namespace {

constexpr unsigned kFullMask = 0xffffffffu;
constexpr int kScanThreads = 1024;
constexpr unsigned long long kNoBadLength = ~0ULL;

struct ChunkTotals {
    long long n_chunks, frames_kept, frames_deleted, pad_frames, sum_t;
    unsigned long long first_bad;
    int t_max, longest_chunk;
};

// chunks of a sequence of t frames, and the frames they keep
__device__ __forceinline__ int chunk_count(int t, int c, unsigned tail) { return tail ? t / c : (t + c - 1) / c; }

__global__ void __launch_bounds__(kScanThreads) kc_scan(const int32_t* __restrict__ lengths, int64_t n, int32_t c, uint32_t tail,
                                                        int64_t* __restrict__ seq_off /*[n] or null*/,
                                                        int64_t* __restrict__ chunk_base /*[n + 1] or null*/,
                                                        ChunkTotals* __restrict__ totals)
{
    __shared__ long long warp_a[kScanThreads / 32], warp_b[kScanThreads / 32];
    __shared__ long long carry_a, carry_b;   // frames and chunks before the current group of sequences
    __shared__ unsigned long long bad_sh;
    __shared__ int max_sh;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { carry_a = 0; carry_b = 0; bad_sh = kNoBadLength; max_sh = 0; }
    __syncthreads();
    int my_max = 0;
    for (int64_t base = 0; base < n; base += kScanThreads) {
        const int64_t i = base + threadIdx.x;
        long long a = 0, b = 0;
        if (i < n) {
            const int t = lengths[i];
            if (t < 1) atomicMin(&bad_sh, (unsigned long long)i);
            else { a = t; b = chunk_count(t, c, tail); my_max = max(my_max, t); }
        }
        long long ia = a, ib = b;  // inclusive scans inside the warp
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const long long ua = __shfl_up_sync(kFullMask, ia, d), ub = __shfl_up_sync(kFullMask, ib, d);
            if (lane >= d) { ia += ua; ib += ub; }
        }
        if (lane == 31) { warp_a[warp] = ia; warp_b[warp] = ib; }
        __syncthreads();
        if (warp == 0) {
            long long wa = warp_a[lane], wb = warp_b[lane];
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const long long ua = __shfl_up_sync(kFullMask, wa, d), ub = __shfl_up_sync(kFullMask, wb, d);
                if (lane >= d) { wa += ua; wb += ub; }
            }
            warp_a[lane] = wa; warp_b[lane] = wb;
        }
        __syncthreads();
        const long long before_a = carry_a + (warp ? warp_a[warp - 1] : 0) + (ia - a);
        const long long before_b = carry_b + (warp ? warp_b[warp - 1] : 0) + (ib - b);
        if (i < n) {
            if (seq_off) seq_off[i] = before_a;
            if (chunk_base) chunk_base[i] = before_b;
        }
        __syncthreads();
        if (threadIdx.x == 0) { carry_a += warp_a[kScanThreads / 32 - 1]; carry_b += warp_b[kScanThreads / 32 - 1]; }
        __syncthreads();
    }
    atomicMax(&max_sh, my_max);
    __syncthreads();
    if (threadIdx.x == 0) {
        if (chunk_base) chunk_base[n] = carry_b;
        ChunkTotals t;
        t.sum_t = carry_a;
        t.n_chunks = carry_b;
        t.first_bad = bad_sh;
        t.t_max = max_sh;
        // kept frames: everything, or the full chunks only; padding: what the kept chunks lack of c frames each
        t.frames_kept = tail ? carry_b * c : carry_a;
        t.frames_deleted = carry_a - t.frames_kept;
        t.pad_frames = carry_b * c - t.frames_kept;
        t.longest_chunk = carry_b == 0 ? 0 : (tail ? c : min(c, max_sh));
        *totals = t;
    }
}

__device__ __forceinline__ uint64_t mix64(uint64_t x)
{   // 64-bit finaliser of MurmurHash3 (Appleby, public domain)
    x ^= x >> 33; x *= 0xFF51AFD7ED558CCDULL; x ^= x >> 33; x *= 0xC4CEB9FE1A85EC53ULL; x ^= x >> 33;
    return x;
}

__global__ void kc_header(PlanHeader* h, const ChunkTotals* __restrict__ totals, int32_t c, uint32_t tail, int64_t expected)
{
    if (threadIdx.x || blockIdx.x) return;
    const ChunkTotals t = *totals;
    memset(h, 0, sizeof *h);
    h->n = t.n_chunks; h->n_blocks = t.n_chunks; h->sum_t = t.sum_t;
    h->first_bad = t.first_bad;
    h->t_block = c; h->t_max = t.longest_chunk;
    h->max_segs = t.n_chunks ? 1 : 0;
    h->policy = 3u + tail;
    h->status = t.first_bad != kNoBadLength ? BLOAD_ERR_LENGTH : (t.n_chunks != expected ? BLOAD_ERR_ARG : BLOAD_OK);
}

__global__ void __launch_bounds__(256) kc_tables(PlanView pv, const int32_t* __restrict__ lengths, int64_t n, int32_t c,
                                                 const int64_t* __restrict__ seq_off, const int64_t* __restrict__ chunk_base,
                                                 int32_t* __restrict__ chunk_seq, int32_t* __restrict__ chunk_first)
{
    if (pv.hdr->status != BLOAD_OK) return;
    const int64_t m = pv.hdr->n;
    unsigned long long term = 0;
    for (int64_t j = (int64_t)blockIdx.x * 256 + threadIdx.x; j < m; j += (int64_t)gridDim.x * 256) {
        // the sequence i with chunk_base[i] <= j < chunk_base[i + 1]
        int64_t lo = 0, hi = n;  // invariant: chunk_base[lo] <= j < chunk_base[hi]
        while (hi - lo > 1) {
            const int64_t mid = (lo + hi) >> 1;
            if (chunk_base[mid] <= j) lo = mid; else hi = mid;
        }
        const int first = (int)(j - chunk_base[lo]) * c;
        const int len = min(c, lengths[lo] - first);
        const int64_t frame = seq_off[lo] + first;
        const int jj = (int)j;
        pv.offsets[j] = frame;
        pv.seg_seq[j] = jj; pv.seg_block[j] = jj; pv.seg_start[j] = 0; pv.seg_src[j] = frame;
        pv.block_seg_begin[j] = jj; pv.block_fill[j] = len;
        pv.seq_block[j] = jj; pv.seq_start[j] = 0;
        if (chunk_seq) chunk_seq[j] = (int)lo;
        if (chunk_first) chunk_first[j] = first;
        term += mix64((((uint64_t)(uint32_t)jj << 32) | 0u) * 0x9E3779B97F4A7C15ULL + (uint64_t)(uint32_t)jj);
        if (j == m - 1) { pv.offsets[m] = pv.hdr->sum_t; pv.block_seg_begin[m] = (int)m; }
    }
#pragma unroll
    for (int d = 16; d; d >>= 1) term += __shfl_xor_sync(kFullMask, term, d);
    if ((threadIdx.x & 31) == 0 && term) atomicAdd(&pv.hdr->checksum, term);
}

__global__ void kc_finish(PlanHeader* h)
{
    if (threadIdx.x == 0 && blockIdx.x == 0 && h->status == BLOAD_OK) h->magic = kPlanMagic;
}

struct ChunkWork { ChunkTotals* totals; int64_t* seq_off; int64_t* chunk_base; };
size_t chunk_work_layout(int64_t n, void* base, ChunkWork* w)
{
    const size_t o_tot = 0, o_off = kAlign, o_base = o_off + align_up(sizeof(int64_t) * (size_t)n);
    const size_t total = o_base + align_up(sizeof(int64_t) * ((size_t)n + 1));
    if (w) {
        char* b = static_cast<char*>(base);
        w->totals = reinterpret_cast<ChunkTotals*>(b + o_tot);
        w->seq_off = reinterpret_cast<int64_t*>(b + o_off);
        w->chunk_base = reinterpret_cast<int64_t*>(b + o_base);
    }
    return total;
}

inline bool aligned_to(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_chunk_args(const int32_t* d_lengths, int64_t n, int32_t t_chunk, uint32_t tail, const void* d_work, size_t work_bytes)
{
    if (!d_lengths || !d_work) return BLOAD_ERR_NULL;
    if (n < 1 || n > 0x7fffffffLL || t_chunk < 1 || tail > BLOAD_CHUNKS_DROP_TAIL) return BLOAD_ERR_ARG;
    if (t_chunk > BLOAD_MAX_T_BLOCK) return BLOAD_ERR_UNSUPPORTED;
    if (work_bytes < chunk_work_layout(n, nullptr, nullptr)) return BLOAD_ERR_WORKSPACE;
    if (!aligned_to(d_work, kAlign) || !aligned_to(d_lengths, 4)) return BLOAD_ERR_ALIGN;
    return BLOAD_OK;
}

void fill_chunk_info(bload_chunk_info_t* out, const ChunkTotals& t, int64_t n, int32_t t_chunk, uint32_t tail)
{
    out->n = n; out->t_chunk = t_chunk; out->tail = tail;
    out->n_chunks = t.n_chunks; out->frames_kept = t.frames_kept; out->frames_deleted = t.frames_deleted;
    out->pad_frames = t.pad_frames; out->sum_t = t.sum_t; out->t_max = t.t_max;
    out->first_bad_index = t.first_bad == kNoBadLength ? -1 : (int64_t)t.first_bad;
    out->status = t.first_bad == kNoBadLength ? BLOAD_OK : BLOAD_ERR_LENGTH;
}

}  // namespace

}  // namespace bload

using namespace bload;

extern "C" {

size_t bload_chunk_work_bytes(int64_t n) { return n < 1 ? 0 : chunk_work_layout(n, nullptr, nullptr); }

int bload_chunk_count(const int32_t* d_lengths, int64_t n, int32_t t_chunk, uint32_t tail, void* d_work, size_t work_bytes,
                      void* stream, bload_chunk_info_t* out)
{
    if (!out) return BLOAD_ERR_NULL;
    memset(out, 0, sizeof *out);
    out->first_bad_index = -1;
    auto fail = [&](int rc) { out->status = rc; return rc; };
    int rc = check_chunk_args(d_lengths, n, t_chunk, tail, d_work, work_bytes);
    if (rc) return fail(rc);
    ChunkWork w;
    chunk_work_layout(n, d_work, &w);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    count_launches(1);
    kc_scan<<<1, kScanThreads, 0, st>>>(d_lengths, n, t_chunk, tail, nullptr, nullptr, w.totals);
    ChunkTotals t;
    cudaError_t ce = cudaPeekAtLastError();
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&t, w.totals, sizeof t, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return fail(BLOAD_ERR_CUDA); }
    fill_chunk_info(out, t, n, t_chunk, tail);
    return out->status;
}

int bload_plan_chunks(const int32_t* d_lengths, int64_t n, int32_t t_chunk, uint32_t tail, int64_t n_chunks, void* d_plan,
                      size_t plan_bytes, void* d_work, size_t work_bytes, int32_t* d_chunk_seq, int32_t* d_chunk_first,
                      void* stream, bload_plan_info_t* info)
{
    if (!info) return BLOAD_ERR_NULL;
    memset(info, 0, sizeof *info);
    info->first_bad_index = -1;
    info->n = n_chunks; info->t_block = t_chunk; info->policy = BLOAD_POLICY_CHUNKS_KEEP_TAIL + tail;
    auto fail = [&](int rc) { info->status = rc; return rc; };
    int rc = check_chunk_args(d_lengths, n, t_chunk, tail, d_work, work_bytes);
    if (rc) return fail(rc);
    if (!d_plan) return fail(BLOAD_ERR_NULL);
    if (n_chunks < 1 || n_chunks > 0x7fffffffLL) return fail(BLOAD_ERR_ARG);
    bload_sizes_t sz;
    plan_layout(n_chunks, &sz);
    if (plan_bytes < sz.plan_bytes) return fail(BLOAD_ERR_WORKSPACE);
    if (!aligned_to(d_plan, kAlign) || !aligned_to(d_chunk_seq, 4) || !aligned_to(d_chunk_first, 4)) return fail(BLOAD_ERR_ALIGN);
    ChunkWork w;
    chunk_work_layout(n, d_work, &w);
    PlanView pv = plan_view(d_plan, n_chunks);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    count_launches(4);
    kc_scan<<<1, kScanThreads, 0, st>>>(d_lengths, n, t_chunk, tail, w.seq_off, w.chunk_base, w.totals);
    kc_header<<<1, 32, 0, st>>>(pv.hdr, w.totals, t_chunk, tail, n_chunks);
    const int64_t want = (n_chunks + 255) / 256, cap = (int64_t)device_info().sm_count * 32;
    kc_tables<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(pv, d_lengths, n, t_chunk, w.seq_off, w.chunk_base,
                                                                   d_chunk_seq, d_chunk_first);
    kc_finish<<<1, 32, 0, st>>>(pv.hdr);
    PlanHeader h;
    cudaError_t ce = cudaPeekAtLastError();
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h, pv.hdr, sizeof h, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return fail(BLOAD_ERR_CUDA); }
    info->status = h.status;
    info->n = h.n; info->n_blocks = h.n_blocks; info->sum_t = h.sum_t; info->t_max = h.t_max;
    info->first_bad_index = h.first_bad == ~0ULL ? -1 : (int64_t)h.first_bad;
    info->checksum = h.checksum;
    info->max_segs_per_block = h.max_segs;
    info->n_source = (uint32_t)n;
    if (h.status == BLOAD_OK && h.magic != kPlanMagic) return fail(BLOAD_ERR_PLAN);
    return info->status;
}

}  // extern "C"

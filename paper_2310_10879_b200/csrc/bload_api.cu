// C ABI of libbload: argument checks, buffer layouts, launches.  See include/bload.h.
#include <string.h>

#include <atomic>
#include <mutex>
#include <vector>

#include "bload_debug.cuh"
#include "bload_internal.cuh"

namespace bload {

#ifdef BLOAD_DEBUG
namespace dbg {
// every translation unit that holds checked kernels adds its reader here (during static initialisation)
static std::vector<void (*)(unsigned long long[4], bool)>& collectors()
{
    static std::vector<void (*)(unsigned long long[4], bool)> v;
    return v;
}
void register_collector(void (*fn)(unsigned long long[4], bool)) { collectors().push_back(fn); }
}  // namespace dbg
#endif

void plan_layout(int64_t n, bload_sizes_t* s)
{
    size_t off = kHeaderBytes;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes); return o; };
    const size_t un = (size_t)n;
    s->max_blocks = n;
    s->off_offsets = take(sizeof(int64_t) * (un + 1));
    s->off_seg_seq = take(sizeof(int32_t) * un);
    s->off_seg_block = take(sizeof(int32_t) * un);
    s->off_seg_start = take(sizeof(int32_t) * un);
    s->off_seg_src = take(sizeof(int64_t) * un);
    s->off_block_seg_begin = take(sizeof(int32_t) * (un + 1));
    s->off_block_fill = take(sizeof(int32_t) * un);
    s->off_seq_block = take(sizeof(int32_t) * un);
    s->off_seq_start = take(sizeof(int32_t) * un);
    s->plan_bytes = off;
}

PlanView plan_view(void* d_plan, int64_t n)
{
    bload_sizes_t s;
    plan_layout(n, &s);
    char* b = static_cast<char*>(d_plan);
    PlanView v;
    v.hdr = reinterpret_cast<PlanHeader*>(b);
    v.offsets = reinterpret_cast<int64_t*>(b + s.off_offsets);
    v.seg_seq = reinterpret_cast<int32_t*>(b + s.off_seg_seq);
    v.seg_block = reinterpret_cast<int32_t*>(b + s.off_seg_block);
    v.seg_start = reinterpret_cast<int32_t*>(b + s.off_seg_start);
    v.seg_src = reinterpret_cast<int64_t*>(b + s.off_seg_src);
    v.block_seg_begin = reinterpret_cast<int32_t*>(b + s.off_block_seg_begin);
    v.block_fill = reinterpret_cast<int32_t*>(b + s.off_block_fill);
    v.seq_block = reinterpret_cast<int32_t*>(b + s.off_seq_block);
    v.seq_start = reinterpret_cast<int32_t*>(b + s.off_seq_start);
    return v;
}

static std::atomic<long long> g_launches{0};
void count_launches(int k) { g_launches.fetch_add(k, std::memory_order_relaxed); }

namespace {
constexpr int kMaxDevices = 64, kMaxOptIns = 32;
std::mutex g_dev_mu;
std::atomic<int> g_dev_known[kMaxDevices];
DeviceInfo g_dev_info[kMaxDevices];
struct OptIn { std::atomic<const void*> kernel; std::atomic<int> bytes; };
OptIn g_opt_in[kMaxDevices][kMaxOptIns];
}  // namespace

static thread_local const char* g_last_kernel[kCopyCalls] = {nullptr, nullptr, nullptr, nullptr, nullptr};
void note_copy_kernel(int call, const char* name) { if (call >= 0 && call < kCopyCalls) g_last_kernel[call] = name; }

DeviceInfo device_info()
{
    DeviceInfo fallback{148, 228 * 1024};
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { (void)cudaGetLastError(); return fallback; }
    if (g_dev_known[dev].load(std::memory_order_acquire)) return g_dev_info[dev];
    std::lock_guard<std::mutex> lock(g_dev_mu);
    if (!g_dev_known[dev].load(std::memory_order_relaxed)) {
        DeviceInfo d = fallback;
        int v = 0;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && v > 0) d.sm_count = v;
        if (cudaDeviceGetAttribute(&v, cudaDevAttrMaxSharedMemoryPerMultiprocessor, dev) == cudaSuccess && v > 0) d.smem_per_sm = v;
        (void)cudaGetLastError();
        g_dev_info[dev] = d;
        g_dev_known[dev].store(1, std::memory_order_release);
    }
    return g_dev_info[dev];
}

cudaError_t opt_in_shared_memory(const void* kernel, int bytes)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    OptIn* row = g_opt_in[dev];
    for (int i = 0; i < kMaxOptIns; ++i) {
        const void* k = row[i].kernel.load(std::memory_order_acquire);
        if (k == kernel && row[i].bytes.load(std::memory_order_relaxed) >= bytes) return cudaSuccess;
        if (!k) break;
    }
    std::lock_guard<std::mutex> lock(g_dev_mu);
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes);
    if (e != cudaSuccess) return e;
    for (int i = 0; i < kMaxOptIns; ++i) {
        const void* k = row[i].kernel.load(std::memory_order_relaxed);
        if (k == kernel || !k) {
            row[i].bytes.store(bytes, std::memory_order_relaxed);
            row[i].kernel.store(kernel, std::memory_order_release);
            break;
        }
    }
    return cudaSuccess;  // a full table only means the attribute is set again next time
}

namespace {
thread_local bool g_timing = false;
thread_local bool g_have_times = false;
thread_local float g_stage_ms[4] = {0, 0, 0, 0};
thread_local bool g_have_epoch_times = false;
thread_local float g_epoch_ms[5] = {0, 0, 0, 0, 0};

// Events of bload_epoch, kept per host thread and device between calls: creating and destroying up to a hundred
// events per call was a visible share of a short epoch.  Every call synchronises both of its streams before it
// returns, so all events of the pool are complete then and can be recorded again by the next call.  The pool is
// never destroyed (at thread exit the CUDA context may already be gone).
struct EventPool {
    int dev = -1;
    std::vector<cudaEvent_t> plain, timed;
    size_t used_plain = 0, used_timed = 0;
    cudaEvent_t take(bool with_timing)
    {
        std::vector<cudaEvent_t>& v = with_timing ? timed : plain;
        size_t& used = with_timing ? used_timed : used_plain;
        if (used == v.size()) {
            cudaEvent_t e = nullptr;
            if (cudaEventCreateWithFlags(&e, with_timing ? cudaEventDefault : cudaEventDisableTiming) != cudaSuccess) return nullptr;
            v.push_back(e);
        }
        return v[used++];
    }
    void begin_call()
    {
        int d = -1;
        if (cudaGetDevice(&d) != cudaSuccess) d = -1;
        if (d != dev) { plain.clear(); timed.clear(); dev = d; }  // events belong to the device they were made on
        used_plain = used_timed = 0;
    }
};
thread_local EventPool* g_events = nullptr;

inline bool aligned(const void* p, uintptr_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

int check_sizes(int64_t n, int32_t t_block)
{
    if (n < 1 || n > 0x7fffffffLL || t_block < 1) return BLOAD_ERR_ARG;
    if (t_block > BLOAD_MAX_T_BLOCK) return BLOAD_ERR_UNSUPPORTED;
    return BLOAD_OK;
}

int check_plan_args(const void* d_plan, const bload_plan_info_t* info, int64_t frame_bytes, int64_t block_begin,
                    int64_t block_count)
{
    if (!d_plan || !info) return BLOAD_ERR_NULL;
    if (info->status != BLOAD_OK || info->n < 1 || info->t_block < 1 || info->n_blocks < 1) return BLOAD_ERR_PLAN;
    if (frame_bytes < 1 || block_begin < 0 || block_count < 0) return BLOAD_ERR_ARG;
    if (block_begin + block_count > 0x7fffffffLL) return BLOAD_ERR_ARG;
    if (!aligned(d_plan, kAlign)) return BLOAD_ERR_ALIGN;
    return BLOAD_OK;
}
}  // namespace

}  // namespace bload

using namespace bload;

extern "C" {

int bload_version(void) { return 1; }

int64_t bload_kernel_launches(void) { return (int64_t)g_launches.load(std::memory_order_relaxed); }

int bload_debug_status(uint64_t out[4], int clear)
{
    if (!out) return BLOAD_ERR_NULL;
    out[0] = out[1] = out[2] = out[3] = 0;
#ifdef BLOAD_DEBUG
    if (cudaDeviceSynchronize() != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    unsigned long long s[4] = {0, 0, 0, 0};
    for (auto fn : dbg::collectors()) fn(s, clear != 0);
    for (int i = 0; i < 4; ++i) out[i] = s[i];
    return BLOAD_OK;
#else
    (void)clear;
    return BLOAD_ERR_UNSUPPORTED;
#endif
}

int64_t bload_bulk_copy_timeouts(void) { return (int64_t)bulk_copy_timeouts(); }

const char* bload_last_copy_kernel(int which)
{
    if (which < 0 || which >= kCopyCalls || !g_last_kernel[which]) return "";
    return g_last_kernel[which];
}

const char* bload_strerror(int code)
{
    switch (code) {
        case BLOAD_OK: return "ok";
        case BLOAD_ERR_NULL: return "a required pointer is NULL";
        case BLOAD_ERR_ARG: return "argument out of range";
        case BLOAD_ERR_LENGTH: return "a sequence length is outside [1, t_block]";
        case BLOAD_ERR_WORKSPACE: return "plan or work buffer too small";
        case BLOAD_ERR_ALIGN: return "device pointer not aligned as required";
        case BLOAD_ERR_UNSUPPORTED: return "unsupported t_block or policy";
        case BLOAD_ERR_CUDA: return "CUDA call failed";
        case BLOAD_ERR_TIMEOUT: return "bounded device wait expired";
        case BLOAD_ERR_PLAN: return "plan is missing, unfinished or failed";
        default: return "unknown error code";
    }
}

int bload_plan_sizes(int64_t n, int32_t t_block, bload_sizes_t* out)
{
    if (!out) return BLOAD_ERR_NULL;
    memset(out, 0, sizeof *out);
    int rc = check_sizes(n, t_block);
    if (rc) return rc;
    plan_layout(n, out);
    // policy 2 and bload_epoch (policy 0) place their extra scratch behind the common part; they never run together
    const size_t extra_bfd = bfd_layout(n, t_block, nullptr, nullptr), extra_epoch = epoch_layout(t_block, nullptr, nullptr);
    out->work_bytes = work_layout(n, t_block, nullptr, nullptr) + (extra_bfd > extra_epoch ? extra_bfd : extra_epoch);
    return BLOAD_OK;
}

int bload_set_plan_timing(int enable)
{
    g_timing = enable != 0;
    return BLOAD_OK;
}

int bload_plan_stage_times(float out_ms[4])
{
    if (!out_ms) return BLOAD_ERR_NULL;
    if (!g_have_times) return BLOAD_ERR_PLAN;
    for (int i = 0; i < 4; ++i) out_ms[i] = g_stage_ms[i];
    return BLOAD_OK;
}

int bload_plan(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy, void* d_plan,
               size_t plan_bytes, void* d_work, size_t work_bytes, void* stream, bload_plan_info_t* info)
{
    if (!info) return BLOAD_ERR_NULL;
    memset(info, 0, sizeof *info);
    info->first_bad_index = -1;
    info->n = n; info->t_block = t_block; info->seed = seed; info->policy = policy;
    auto fail = [&](int rc) { info->status = rc; return rc; };
    if (!d_lengths || !d_plan || !d_work) return fail(BLOAD_ERR_NULL);
    int rc = check_sizes(n, t_block);
    if (rc) return fail(rc);
    if (policy > BLOAD_POLICY_BEST_FIT_DECREASING) return fail(BLOAD_ERR_UNSUPPORTED);
    if (policy == BLOAD_POLICY_UNIFORM_LENGTHS && n >= (1LL << 26)) return fail(BLOAD_ERR_UNSUPPORTED);
    bload_sizes_t sz;
    plan_layout(n, &sz);
    WorkView wv;
    BfdView bv;
    size_t need_work = work_layout(n, t_block, d_work, &wv);  // the size bload_plan_sizes reports covers every policy
    {
        const size_t extra_bfd = bfd_layout(n, t_block, static_cast<char*>(d_work) + need_work, &bv);
        const size_t extra_epoch = epoch_layout(t_block, nullptr, nullptr);
        need_work += extra_bfd > extra_epoch ? extra_bfd : extra_epoch;
    }
    if (plan_bytes < sz.plan_bytes || work_bytes < need_work) return fail(BLOAD_ERR_WORKSPACE);
    if (!aligned(d_plan, kAlign) || !aligned(d_work, kAlign) || !aligned(d_lengths, 4)) return fail(BLOAD_ERR_ALIGN);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlanView pv = plan_view(d_plan, n);
    cudaEvent_t ev[5];
    bool timing = g_timing;
    if (timing)
        for (int i = 0; i < 5; ++i)
            if (cudaEventCreate(&ev[i]) != cudaSuccess) { timing = false; break; }
    cudaError_t ce = launch_plan(d_lengths, n, t_block, seed, policy, pv, wv, st, timing ? ev : nullptr, &bv);
    PlanHeader h;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h, pv.hdr, sizeof h, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (timing) {
        if (ce == cudaSuccess) {
            for (int i = 0; i < 4; ++i) cudaEventElapsedTime(&g_stage_ms[i], ev[i], ev[i + 1]);
            g_have_times = true;
        }
        for (int i = 0; i < 5; ++i) cudaEventDestroy(ev[i]);
    }
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return fail(BLOAD_ERR_CUDA); }

    info->status = h.status;
    info->n_blocks = h.n_blocks;
    info->sum_t = h.sum_t;
    info->t_max = h.t_max;
    info->first_bad_index = h.first_bad == ~0ULL ? -1 : (int64_t)h.first_bad;
    info->checksum = h.checksum;
    info->max_segs_per_block = h.max_segs;
    if (h.status == BLOAD_OK && h.magic != kPlanMagic) return fail(BLOAD_ERR_PLAN);
    return info->status;
}

int bload_plan_async(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy, void* d_plan,
                     size_t plan_bytes, void* d_work, size_t work_bytes, void* stream)
{
    if (!d_lengths || !d_plan || !d_work) return BLOAD_ERR_NULL;
    int rc = check_sizes(n, t_block);
    if (rc) return rc;
    if (policy > BLOAD_POLICY_BEST_FIT_DECREASING) return BLOAD_ERR_UNSUPPORTED;
    if (policy == BLOAD_POLICY_UNIFORM_LENGTHS && n >= (1LL << 26)) return BLOAD_ERR_UNSUPPORTED;
    bload_sizes_t sz;
    plan_layout(n, &sz);
    WorkView wv;
    BfdView bv;
    size_t need_work = work_layout(n, t_block, d_work, &wv);  // the size bload_plan_sizes reports covers every policy
    {
        const size_t extra_bfd = bfd_layout(n, t_block, static_cast<char*>(d_work) + need_work, &bv);
        const size_t extra_epoch = epoch_layout(t_block, nullptr, nullptr);
        need_work += extra_bfd > extra_epoch ? extra_bfd : extra_epoch;
    }
    if (plan_bytes < sz.plan_bytes || work_bytes < need_work) return BLOAD_ERR_WORKSPACE;
    if (!aligned(d_plan, kAlign) || !aligned(d_work, kAlign) || !aligned(d_lengths, 4)) return BLOAD_ERR_ALIGN;
    cudaError_t ce = launch_plan(d_lengths, n, t_block, seed, policy, plan_view(d_plan, n), wv,
                                 static_cast<cudaStream_t>(stream), nullptr, &bv);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_plan_finish(const void* d_plan, void* stream, bload_plan_info_t* info)
{
    if (!info) return BLOAD_ERR_NULL;
    memset(info, 0, sizeof *info);
    info->first_bad_index = -1;
    auto fail = [&](int rc) { info->status = rc; return rc; };
    if (!d_plan) return fail(BLOAD_ERR_NULL);
    if (!aligned(d_plan, kAlign)) return fail(BLOAD_ERR_ALIGN);
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlanHeader h;
    cudaError_t ce = cudaMemcpyAsync(&h, d_plan, sizeof h, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return fail(BLOAD_ERR_CUDA); }
    info->n = h.n; info->t_block = h.t_block; info->seed = h.seed; info->policy = h.policy;
    info->status = h.status;
    info->n_blocks = h.n_blocks;
    info->sum_t = h.sum_t;
    info->t_max = h.t_max;
    info->first_bad_index = h.first_bad == ~0ULL ? -1 : (int64_t)h.first_bad;
    info->checksum = h.checksum;
    info->max_segs_per_block = h.max_segs;
    if (h.status == BLOAD_OK && h.magic != kPlanMagic) return fail(BLOAD_ERR_PLAN);
    return info->status;
}

int bload_epoch_stage_times(float out_ms[5])
{
    if (!out_ms) return BLOAD_ERR_NULL;
    if (!g_have_epoch_times) return BLOAD_ERR_PLAN;
    for (int i = 0; i < 5; ++i) out_ms[i] = g_epoch_ms[i];
    return BLOAD_OK;
}

int bload_epoch(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, void* d_plan, size_t plan_bytes,
                void* d_work, size_t work_bytes, const bload_epoch_io_t* io, void* stream, void* side_stream,
                bload_plan_info_t* info)
{
    if (!info) return BLOAD_ERR_NULL;
    memset(info, 0, sizeof *info);
    info->first_bad_index = -1;
    info->n = n; info->t_block = t_block; info->seed = seed; info->policy = BLOAD_POLICY_UNIFORM_SEQUENCES;
    auto fail = [&](int rc) { info->status = rc; return rc; };
    if (!d_lengths || !d_plan || !d_work || !io) return fail(BLOAD_ERR_NULL);
    int rc = check_sizes(n, t_block);
    if (rc) return fail(rc);
    const bool do_pack = io->d_dense != nullptr, do_unpack = io->d_dense_out != nullptr;
    const bool do_meta = io->d_seq_id || io->d_pos || io->d_reset || io->d_valid;
    if (do_pack && !io->d_store) return fail(BLOAD_ERR_NULL);
    if (do_unpack && !io->d_ragged_out) return fail(BLOAD_ERR_NULL);
    if ((do_pack && io->frame_bytes < 1) || (do_unpack && io->out_frame_bytes < 1) || io->block_capacity < 1 ||
        io->block_capacity > 0x7fffffffLL || io->chunks > kMaxEpochChunks)
        return fail(BLOAD_ERR_ARG);
    if (do_pack && (!aligned(io->d_dense, 16) || !aligned(io->d_store, 16))) return fail(BLOAD_ERR_ALIGN);
    if (do_unpack && (!aligned(io->d_dense_out, 16) || !aligned(io->d_ragged_out, 16))) return fail(BLOAD_ERR_ALIGN);
    if (!aligned(io->d_seq_id, 4) || !aligned(io->d_pos, 4)) return fail(BLOAD_ERR_ALIGN);
    bload_sizes_t sz;
    plan_layout(n, &sz);
    WorkView wv;
    EpochView ev;
    size_t need_work = work_layout(n, t_block, d_work, &wv);
    {
        const size_t extra_epoch = epoch_layout(t_block, static_cast<char*>(d_work) + need_work, &ev);
        const size_t extra_bfd = bfd_layout(n, t_block, nullptr, nullptr);
        need_work += extra_bfd > extra_epoch ? extra_bfd : extra_epoch;  // the one size bload_plan_sizes reports
    }
    if (plan_bytes < sz.plan_bytes || work_bytes < need_work) return fail(BLOAD_ERR_WORKSPACE);
    if (!aligned(d_plan, kAlign) || !aligned(d_work, kAlign) || !aligned(d_lengths, 4)) return fail(BLOAD_ERR_ALIGN);

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    cudaStream_t side = side_stream ? static_cast<cudaStream_t>(side_stream) : st;
    PlanView pv = plan_view(d_plan, n);
    const int32_t cap = (int32_t)io->block_capacity;
    // Chunks of about 1,800 draws on average, at most 10: the first chunk delays the copies and the last chunk's copies are
    // an exposed tail, but every chunk costs launches and the hand-over of the fill rule's tables (about 40 us).  Chunks
    // chosen by the caller are equal.  The library's own grow geometrically (each 1.25 times the one before): the copies
    // of a chunk take longer than its draws (they are what the step waits for), so a short first chunk starts them early
    // and later chunks can be long without the copying stream running dry.  Measured on 20,000 heavy-tailed lengths, ms
    // per step: equal chunks 1: 7.8, 4: 5.4, 8: 5.13, 10-12: 5.10, 16: 5.17, 32: 5.6; growing chunks 12 x 1.1: 4.97,
    // 12 x 1.2: 4.92, 12 x 1.3: 4.91, 12 x 1.4: 5.13, 12 x 2.0: 5.93, 8 x 1.2: 4.90, 8 x 1.4: 5.11, 16 x 1.15: 4.92,
    // 10 x 1.25: 4.87.
    constexpr int kOwnChunks = 10;
    constexpr double kChunkGrowth = 1.25;
    int chunks = (int)(n / 1800);
    if (chunks < 1) chunks = 1;
    if (chunks > kOwnChunks) chunks = kOwnChunks;
    if (io->chunks) chunks = io->chunks;
    double chunk_end[kMaxEpochChunks];  // where the chunks end, as fractions of the draws
    {
        const double g = io->chunks ? 1.0 : kChunkGrowth;
        double total = 0.0, w = 1.0;
        for (int c = 0; c < chunks; ++c) { total += w; chunk_end[c] = total; w *= g; }
        for (int c = 0; c < chunks; ++c) chunk_end[c] /= total;
    }
    const bool timing = g_timing;
    g_have_epoch_times = false;

    // events: one per chunk to hand its blocks to the side stream, one to join; with timing, 2 + 5 more per chunk
    if (!g_events) g_events = new EventPool;
    g_events->begin_call();
    auto new_event = [&](bool timed) -> cudaEvent_t { return g_events->take(timed); };
    struct ChunkEv { cudaEvent_t f0, f1, ready, t0, t1, t2, t3, t4; } ce_[kMaxEpochChunks];

    cudaError_t ce = cudaMemsetAsync(ev.resume, 0, sizeof(FillResume), st);
    int32_t* sorted_id = nullptr;
    if (ce == cudaSuccess)
        ce = launch_plan_front(d_lengths, n, t_block, seed, BLOAD_POLICY_UNIFORM_SEQUENCES, pv, wv, st, &sorted_id);
    const int64_t dense_total = do_unpack ? io->block_capacity * (int64_t)t_block * io->out_frame_bytes : 0;
    for (int c = 0; c < chunks && ce == cudaSuccess; ++c) {
        ChunkEv& E = ce_[c];
        E = ChunkEv{};
        if (timing) { E.f0 = new_event(true); E.f1 = new_event(true); }
        E.ready = new_event(false);
        if (timing) { E.t0 = new_event(true); E.t1 = new_event(true); E.t2 = new_event(true); E.t3 = new_event(true); E.t4 = new_event(true); }
        if (!E.ready || (timing && (!E.f0 || !E.f1 || !E.t0 || !E.t1 || !E.t2 || !E.t3 || !E.t4))) { ce = cudaErrorMemoryAllocation; break; }
        const int32_t k_target = c + 1 == chunks ? (int32_t)n : (int32_t)(n * chunk_end[c]);
        if (timing) cudaEventRecord(E.f0, st);
        ce = launch_fill_chunk(pv, wv, ev, n, t_block, k_target, cap, st);
        if (timing) cudaEventRecord(E.f1, st);
        if (ce != cudaSuccess) break;
        cudaEventRecord(E.ready, st);
        if (side != st) cudaStreamWaitEvent(side, E.ready, 0);
        const int32_t* d_blocks = ev.resume->range[c];
        const int32_t* d_draws = ev.resume->draw[c];
        if (timing) cudaEventRecord(E.t0, side);
        ce = launch_tables_chunk(pv, wv, sorted_id, n, d_draws, side);
        if (timing) cudaEventRecord(E.t1, side);
        if (ce == cudaSuccess && do_meta)
            ce = launch_metadata(pv, t_block, 0, 0, io->d_seq_id, io->d_pos, io->d_reset, io->d_valid, side, d_blocks);
        if (timing) cudaEventRecord(E.t2, side);
        if (ce == cudaSuccess && do_pack)
            ce = launch_copy_range(false, pv, t_block, io->frame_bytes, static_cast<const uint8_t*>(io->d_store),
                                   static_cast<uint8_t*>(io->d_dense), 0 /*taken from the plan on the device*/, io->pad_byte, d_blocks, side);
        if (timing) cudaEventRecord(E.t3, side);
        if (ce == cudaSuccess && do_unpack)
            ce = launch_copy_range(true, pv, t_block, io->out_frame_bytes, static_cast<const uint8_t*>(io->d_dense_out),
                                   static_cast<uint8_t*>(io->d_ragged_out), dense_total, 0, d_blocks, side);
        if (timing) cudaEventRecord(E.t4, side);
    }
    // filler blocks between the end of the plan and the end of the caller's buffers, then the plan is complete
    if (ce == cudaSuccess) {
        const int32_t* d_tail = ev.resume->range[kMaxEpochChunks];
        if (do_meta) ce = launch_metadata(pv, t_block, 0, 0, io->d_seq_id, io->d_pos, io->d_reset, io->d_valid, side, d_tail);
        if (ce == cudaSuccess && do_pack)
            ce = launch_copy_range(false, pv, t_block, io->frame_bytes, static_cast<const uint8_t*>(io->d_store),
                                   static_cast<uint8_t*>(io->d_dense), 0, io->pad_byte, d_tail, side);
        if (ce == cudaSuccess) ce = launch_plan_finish(pv, side);
    }
    if (ce == cudaSuccess && side != st) {
        cudaEvent_t join = new_event(false);
        if (!join) ce = cudaErrorMemoryAllocation;
        else { cudaEventRecord(join, side); cudaStreamWaitEvent(st, join, 0); }
    }
    PlanHeader h;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h, pv.hdr, sizeof h, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) {
        (void)cudaGetLastError();
        cudaStreamSynchronize(side); cudaStreamSynchronize(st);  // nothing may still use the events
        return fail(BLOAD_ERR_CUDA);
    }
    if (timing) {
        for (int i = 0; i < 5; ++i) g_epoch_ms[i] = 0.f;
        for (int c = 0; c < chunks; ++c) {
            float ms = 0.f;
            const ChunkEv& E = ce_[c];
            if (cudaEventElapsedTime(&ms, E.f0, E.f1) == cudaSuccess) g_epoch_ms[0] += ms;
            if (cudaEventElapsedTime(&ms, E.t0, E.t1) == cudaSuccess) g_epoch_ms[1] += ms;
            if (cudaEventElapsedTime(&ms, E.t1, E.t2) == cudaSuccess) g_epoch_ms[2] += ms;
            if (cudaEventElapsedTime(&ms, E.t2, E.t3) == cudaSuccess) g_epoch_ms[3] += ms;
            if (cudaEventElapsedTime(&ms, E.t3, E.t4) == cudaSuccess) g_epoch_ms[4] += ms;
        }
        g_have_epoch_times = true;
    }
    info->status = h.status;
    info->n_blocks = h.n_blocks;
    info->sum_t = h.sum_t;
    info->t_max = h.t_max;
    info->first_bad_index = h.first_bad == ~0ULL ? -1 : (int64_t)h.first_bad;
    info->checksum = h.checksum;
    info->max_segs_per_block = h.max_segs;
    if (h.status == BLOAD_OK && h.magic != kPlanMagic) return fail(BLOAD_ERR_PLAN);
    if (h.status == BLOAD_OK && h.n_blocks > io->block_capacity) return BLOAD_ERR_WORKSPACE;  // the plan itself is complete
    return info->status;
}

int bload_pack(const void* d_plan, const bload_plan_info_t* info, const void* d_store, int64_t frame_bytes,
               int64_t block_begin, int64_t block_count, void* d_dense, int32_t* d_seq_id, int32_t* d_pos,
               uint8_t* d_reset, uint8_t* d_valid, uint8_t pad_byte, void* stream)
{
    int rc = check_plan_args(d_plan, info, frame_bytes, block_begin, block_count);
    if (rc) return rc;
    if (block_count == 0) return BLOAD_OK;
    if (d_dense && !d_store) return BLOAD_ERR_NULL;
    if (d_dense && (!aligned(d_dense, 16) || !aligned(d_store, 16))) return BLOAD_ERR_ALIGN;
    if (!aligned(d_seq_id, 4) || !aligned(d_pos, 4)) return BLOAD_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlanView pv = plan_view(const_cast<void*>(d_plan), info->n);
    cudaError_t ce = cudaSuccess;
    const bool want_meta = d_seq_id || d_pos || d_reset || d_valid;
    // a small call for dense blocks and metadata of small frames: one launch does both
    if (want_meta && d_dense &&
        staged_pack_with_metadata(pv, info->t_block, frame_bytes, block_begin, block_count, static_cast<const uint8_t*>(d_store),
                                  static_cast<uint8_t*>(d_dense), d_seq_id, d_pos, d_reset, d_valid,
                                  info->sum_t * frame_bytes, pad_byte, st, info->n, &ce)) {
        if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
        return BLOAD_OK;
    }
    if (want_meta)
        ce = launch_metadata(pv, info->t_block, block_begin, block_count, d_seq_id, d_pos, d_reset, d_valid, st, nullptr, info->n, info->sum_t);
    if (ce == cudaSuccess && d_dense)
        ce = launch_copy(false, pv, info->t_block, frame_bytes, block_begin, block_count,
                         static_cast<const uint8_t*>(d_store), static_cast<uint8_t*>(d_dense), nullptr,
                         info->sum_t * frame_bytes, pad_byte, st, info->n, info->n_blocks, false, want_meta);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_pack_repeat_last(const void* d_plan, const bload_plan_info_t* info, const void* d_store, int64_t frame_bytes,
                           int64_t block_begin, int64_t block_count, void* d_dense, int32_t* d_seq_id, int32_t* d_pos,
                           uint8_t* d_reset, uint8_t* d_valid, uint8_t pad_byte, void* stream)
{
    int rc = bload_pack(d_plan, info, d_store, frame_bytes, block_begin, block_count, d_dense, d_seq_id, d_pos, d_reset,
                        d_valid, pad_byte, stream);
    if (rc || block_count == 0 || !d_dense) return rc;
    cudaError_t ce = launch_repeat_last(plan_view(const_cast<void*>(d_plan), info->n), info->t_block, frame_bytes,
                                        block_begin, block_count, static_cast<uint8_t*>(d_dense),
                                        static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_unpack(const void* d_plan, const bload_plan_info_t* info, const void* d_dense_out, int64_t out_frame_bytes,
                 int64_t block_begin, int64_t block_count, void* d_ragged_out, void* stream)
{
    int rc = check_plan_args(d_plan, info, out_frame_bytes, block_begin, block_count);
    if (rc) return rc;
    if (block_count == 0) return BLOAD_OK;
    if (!d_dense_out || !d_ragged_out) return BLOAD_ERR_NULL;
    if (!aligned(d_dense_out, 16) || !aligned(d_ragged_out, 16)) return BLOAD_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlanView pv = plan_view(const_cast<void*>(d_plan), info->n);
    cudaError_t ce = launch_copy(true, pv, info->t_block, out_frame_bytes, block_begin, block_count, nullptr,
                                 const_cast<uint8_t*>(static_cast<const uint8_t*>(d_dense_out)),
                                 static_cast<uint8_t*>(d_ragged_out), info->sum_t * out_frame_bytes, 0, st, info->n,
                                 info->n_blocks, info->policy == BLOAD_POLICY_CHUNKS_DROP_TAIL);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_var_offsets2d(const int32_t* d_lengths, const int32_t* d_rows, const int32_t* d_row_bytes, int64_t n,
                        int64_t* d_byte_offsets, void* stream, bload_var_info_t* info)
{
    if (!info) return BLOAD_ERR_NULL;
    memset(info, 0, sizeof *info);
    info->first_bad_index = -1;
    if (!d_lengths || !d_row_bytes || !d_byte_offsets) return BLOAD_ERR_NULL;
    if (n < 1 || n >= (1LL << 31)) return BLOAD_ERR_ARG;
    if (!aligned(d_lengths, 4) || !aligned(d_rows, 4) || !aligned(d_row_bytes, 4) || !aligned(d_byte_offsets, 8))
        return BLOAD_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // the tail of the array: [n] total bytes, [n+1] largest row size, [n+2] first bad index, and with rows [n+3] most rows
    cudaError_t ce = launch_var_offsets(d_lengths, d_rows, d_row_bytes, n, d_byte_offsets,
                                        d_rows ? d_byte_offsets + n + 3 : nullptr, st);
    int64_t tail[4] = {0, 0, -1, 1};
    if (ce == cudaSuccess)
        ce = cudaMemcpyAsync(tail, d_byte_offsets + n, (d_rows ? 4 : 3) * sizeof(int64_t), cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    info->total_bytes = tail[0];
    info->max_frame_bytes = tail[1];
    info->first_bad_index = tail[2];
    info->max_rows = tail[3];
    return tail[2] >= 0 ? BLOAD_ERR_ARG : BLOAD_OK;
}

int bload_var_offsets(const int32_t* d_lengths, const int32_t* d_frame_bytes, int64_t n, int64_t* d_byte_offsets,
                      void* stream, bload_var_info_t* info)
{
    return bload_var_offsets2d(d_lengths, nullptr, d_frame_bytes, n, d_byte_offsets, stream, info);
}

namespace {
int copy_var(bool unpack, const void* d_plan, const bload_plan_info_t* info, const void* d_src, const int32_t* d_rows,
             const int32_t* d_row_bytes, const int64_t* d_byte_offsets, int64_t rows_max, int64_t row_stride,
             int64_t block_begin, int64_t block_count, void* d_dst, uint8_t pad_byte, void* stream)
{
    int rc = check_plan_args(d_plan, info, row_stride, block_begin, block_count);
    if (rc) return rc;
    if (info->policy >= BLOAD_POLICY_CHUNKS_KEEP_TAIL) return BLOAD_ERR_UNSUPPORTED;  // sizes are per sequence, chunks are not sequences
    if (rows_max < 1 || rows_max > 0x7fffffffLL) return BLOAD_ERR_ARG;
    if (block_count == 0) return BLOAD_OK;
    if (!d_src || !d_dst || !d_row_bytes || !d_byte_offsets) return BLOAD_ERR_NULL;
    if (!aligned(d_src, 16) || !aligned(d_dst, 16) || !aligned(d_rows, 4) || !aligned(d_row_bytes, 4) ||
        !aligned(d_byte_offsets, 8))
        return BLOAD_ERR_ALIGN;
    cudaError_t ce = launch_copy_var(unpack, plan_view(const_cast<void*>(d_plan), info->n), info->t_block, (int32_t)rows_max,
                                     row_stride, block_begin, block_count, d_rows, d_row_bytes, d_byte_offsets,
                                     static_cast<const uint8_t*>(d_src), static_cast<uint8_t*>(d_dst), pad_byte,
                                     static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}
}  // namespace

int bload_pack_var(const void* d_plan, const bload_plan_info_t* info, const void* d_store, const int32_t* d_frame_bytes,
                   const int64_t* d_byte_offsets, int64_t slot_bytes, int64_t block_begin, int64_t block_count,
                   void* d_dense, uint8_t pad_byte, void* stream)
{
    return copy_var(false, d_plan, info, d_store, nullptr, d_frame_bytes, d_byte_offsets, 1, slot_bytes, block_begin,
                    block_count, d_dense, pad_byte, stream);
}

int bload_unpack_var(const void* d_plan, const bload_plan_info_t* info, const void* d_dense_out,
                     const int32_t* d_frame_bytes, const int64_t* d_byte_offsets, int64_t slot_bytes, int64_t block_begin,
                     int64_t block_count, void* d_ragged_out, void* stream)
{
    return copy_var(true, d_plan, info, d_dense_out, nullptr, d_frame_bytes, d_byte_offsets, 1, slot_bytes, block_begin,
                    block_count, d_ragged_out, 0, stream);
}

int bload_pack_var2d(const void* d_plan, const bload_plan_info_t* info, const void* d_store, const int32_t* d_rows,
                     const int32_t* d_row_bytes, const int64_t* d_byte_offsets, int64_t rows_max, int64_t row_stride,
                     int64_t block_begin, int64_t block_count, void* d_dense, uint8_t pad_byte, void* stream)
{
    if (!d_rows) return BLOAD_ERR_NULL;
    return copy_var(false, d_plan, info, d_store, d_rows, d_row_bytes, d_byte_offsets, rows_max, row_stride, block_begin,
                    block_count, d_dense, pad_byte, stream);
}

int bload_unpack_var2d(const void* d_plan, const bload_plan_info_t* info, const void* d_dense_out, const int32_t* d_rows,
                       const int32_t* d_row_bytes, const int64_t* d_byte_offsets, int64_t rows_max, int64_t row_stride,
                       int64_t block_begin, int64_t block_count, void* d_ragged_out, void* stream)
{
    if (!d_rows) return BLOAD_ERR_NULL;
    return copy_var(true, d_plan, info, d_dense_out, d_rows, d_row_bytes, d_byte_offsets, rows_max, row_stride, block_begin,
                    block_count, d_ragged_out, 0, stream);
}

int bload_carry_prev(const void* d_plan, const bload_plan_info_t* info, const void* d_dense, int64_t frame_bytes,
                     int64_t block_begin, int64_t block_count, void* d_prev, uint8_t fill_byte, void* stream)
{
    int rc = check_plan_args(d_plan, info, frame_bytes, block_begin, block_count);
    if (rc) return rc;
    if (block_count == 0) return BLOAD_OK;
    if (!d_dense || !d_prev) return BLOAD_ERR_NULL;
    if (d_dense == d_prev) return BLOAD_ERR_ARG;
    if (!aligned(d_dense, 16) || !aligned(d_prev, 16)) return BLOAD_ERR_ALIGN;
    cudaError_t ce = launch_carry_prev(plan_view(const_cast<void*>(d_plan), info->n), info->t_block, frame_bytes,
                                       block_begin, block_count, static_cast<const uint8_t*>(d_dense),
                                       static_cast<uint8_t*>(d_prev), fill_byte, static_cast<cudaStream_t>(stream), info->n,
                                       info->sum_t);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_reset_state(const void* d_plan, const bload_plan_info_t* info, int64_t block_begin, int64_t block_count,
                      int32_t slot, void* d_state, int64_t state_bytes, const void* d_init, void* stream)
{
    int rc = check_plan_args(d_plan, info, state_bytes, block_begin, block_count);
    if (rc) return rc;
    if (slot < 0 || slot >= info->t_block) return BLOAD_ERR_ARG;
    if (block_count == 0) return BLOAD_OK;
    if (!d_state) return BLOAD_ERR_NULL;
    if (!aligned(d_init, 16)) return BLOAD_ERR_ALIGN;
    cudaError_t ce = launch_reset_state(plan_view(const_cast<void*>(d_plan), info->n), block_begin, block_count, slot,
                                        static_cast<uint8_t*>(d_state), state_bytes, static_cast<const uint8_t*>(d_init),
                                        static_cast<cudaStream_t>(stream));
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_valid_sum(const void* d_plan, const bload_plan_info_t* info, const float* d_values, int64_t block_begin,
                    int64_t block_count, double* d_block_sum, double* d_total, void* stream)
{
    int rc = check_plan_args(d_plan, info, 1, block_begin, block_count);
    if (rc) return rc;
    if (!d_values || !d_block_sum) return BLOAD_ERR_NULL;
    if (!aligned(d_values, 4) || !aligned(d_block_sum, 8) || !aligned(d_total, 8)) return BLOAD_ERR_ALIGN;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (block_count == 0) {  // an empty range sums to zero over zero frames
        if (d_total && cudaMemsetAsync(d_total, 0, 2 * sizeof(double), st) != cudaSuccess) {
            (void)cudaGetLastError();
            return BLOAD_ERR_CUDA;
        }
        return BLOAD_OK;
    }
    cudaError_t ce = launch_valid_sum(plan_view(const_cast<void*>(d_plan), info->n), info->t_block, block_begin, block_count,
                                      d_values, d_block_sum, d_total, st);
    if (ce != cudaSuccess) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
    return BLOAD_OK;
}

int bload_rank_range(int64_t n_blocks, int32_t world_size, int32_t rank, int32_t batch_blocks, int64_t* out_begin,
                     int64_t* out_count)
{
    if (!out_begin || !out_count) return BLOAD_ERR_NULL;
    *out_begin = 0; *out_count = 0;
    if (n_blocks < 1 || world_size < 1 || rank < 0 || rank >= world_size || batch_blocks < 1) return BLOAD_ERR_ARG;
    const int64_t share = (n_blocks + world_size - 1) / world_size;
    const int64_t per_rank = (share + batch_blocks - 1) / batch_blocks * batch_blocks;
    if (per_rank * world_size > 0x7fffffffLL) return BLOAD_ERR_ARG;
    *out_begin = per_rank * rank;
    *out_count = per_rank;
    return BLOAD_OK;
}

int bload_stats(const bload_plan_info_t* info, bload_stats_t* out)
{
    if (!info || !out) return BLOAD_ERR_NULL;
    memset(out, 0, sizeof *out);
    if (info->status != BLOAD_OK || info->n < 1 || info->t_block < 1 || info->n_blocks < 1 || info->sum_t < 1)
        return BLOAD_ERR_PLAN;
    const int64_t n = info->n, tb = info->t_block, nb = info->n_blocks, tm = info->t_max;
    // frames that sit in blocks: all of the store, except under the chunking strategy that keeps only full chunks
    const int64_t s = info->policy == BLOAD_POLICY_CHUNKS_DROP_TAIL ? nb * tb : info->sum_t;
    out->frames_deleted = info->sum_t - s;
    out->n = n; out->sum_t = s; out->t_max = tm; out->t_block = tb; out->n_blocks = nb;
    out->pad_packed = nb * tb - s;
    out->pad_naive_tmax = n * tm - s;
    out->pad_naive_tblock = n * tb - s;
    out->min_blocks = (s + tb - 1) / tb;
    out->frac_packed = (double)out->pad_packed / (double)(nb * tb);
    out->frac_naive_tmax = tm > 0 ? (double)out->pad_naive_tmax / (double)(n * tm) : 0.0;
    out->frac_naive_tblock = (double)out->pad_naive_tblock / (double)(n * tb);
    out->reduction_vs_tmax = out->pad_packed > 0 ? (double)out->pad_naive_tmax / (double)out->pad_packed : 0.0;
    out->mean_segs_per_block = (double)n / (double)nb;
    out->max_segs_per_block = info->max_segs_per_block;
    return BLOAD_OK;
}

}  // extern "C"

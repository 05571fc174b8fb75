// bload_plan_static: the planner with its scratch memory built into the library image.
//
// Some callers of the planner cannot obtain device memory at the moment they need a plan: a
// data-loading thread that runs beside a training job whose framework has already claimed the
// device's memory for its own caching pool (a fresh cudaMalloc there can fail, and it can stall
// the whole device while the driver serves it), or a latency-sensitive loop that is forbidden to
// call the allocator at all.  For them the scratch buffer that bload_plan takes from the caller
// is replaced here by a fixed array that is part of the loaded library on every GPU.  Nothing in
// this file allocates or frees memory.
#include <string.h>

#include <mutex>

#include "bload_internal.cuh"

namespace {

// The scratch itself.  Every device that loads the library carries these bytes until the process ends.
static __device__ __align__(256) unsigned char g_static_scratch[BLOAD_STATIC_SCRATCH_BYTES];

// In host code the name above is only a handle for the symbol; the address a kernel can use has
// to be asked for, per device, with that device current.
constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_addr[kMaxDevices] = {nullptr};

int scratch_for_current_device(void** out)
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BLOAD_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_addr[dev]) {
        void* p = nullptr;
        cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
        if (e != cudaSuccess || !p) { (void)cudaGetLastError(); return BLOAD_ERR_CUDA; }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return BLOAD_OK;
}

}  // namespace

using namespace bload;

extern "C" int bload_plan_static(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                                 void* d_plan, size_t plan_bytes, void* stream, bload_plan_info_t* info)
{
    if (!info) return BLOAD_ERR_NULL;
    memset(info, 0, sizeof *info);
    info->first_bad_index = -1;
    info->n = n; info->t_block = t_block; info->seed = seed; info->policy = policy;
    auto fail = [&](int rc) { info->status = rc; return rc; };
    if (!d_lengths || !d_plan) return fail(BLOAD_ERR_NULL);
    if (n < 1 || t_block < 1) return fail(BLOAD_ERR_ARG);
    // both readings of the paper's rule run in the common scratch layout; best fit decreasing needs about 40 more
    // bytes per sequence behind it, which this array was not sized for
    if (t_block > BLOAD_MAX_T_BLOCK || policy > BLOAD_POLICY_UNIFORM_LENGTHS) return fail(BLOAD_ERR_UNSUPPORTED);
    // the built-in scratch is a fixed size: larger problems must use bload_plan with a caller buffer
    if (n > BLOAD_STATIC_MAX_N || work_layout(n, t_block, nullptr, nullptr) > (size_t)BLOAD_STATIC_SCRATCH_BYTES)
        return fail(BLOAD_ERR_WORKSPACE);
    bload_sizes_t sz;
    plan_layout(n, &sz);
    if (plan_bytes < sz.plan_bytes) return fail(BLOAD_ERR_WORKSPACE);
    if ((reinterpret_cast<uintptr_t>(d_plan) & (kAlign - 1)) || (reinterpret_cast<uintptr_t>(d_lengths) & 3))
        return fail(BLOAD_ERR_ALIGN);

    void* scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc) return fail(rc);
    WorkView wv;
    work_layout(n, t_block, scratch, &wv);  // every scratch table is fully rewritten by the kernels: nothing to clear

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PlanView pv = plan_view(d_plan, n);
    cudaError_t ce = launch_plan(d_lengths, n, t_block, seed, policy, pv, wv, st, nullptr);
    PlanHeader h;
    if (ce == cudaSuccess) ce = cudaMemcpyAsync(&h, pv.hdr, sizeof h, cudaMemcpyDeviceToHost, st);
    if (ce == cudaSuccess) ce = cudaStreamSynchronize(st);
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

// Bounds checking of the library's own global-memory accesses, compiled in with -DBLOAD_DEBUG (a second library,
// libbload_debug.so: `python -m paper_2310_10879_b200.build --debug`).  It stands in for a memory checker where none
// can be run: before a launch the launcher registers the byte ranges the kernel may read and the ranges it may write;
// every data access of the copy, metadata and table kernels asks first, and an access outside its ranges is SKIPPED
// and recorded -- never trapped, never asserted -- so the context stays usable and the test that provoked it can read
// what happened with bload_debug_status.  Without the flag every hook compiles to nothing.
//
// The registered ranges live in one __device__ variable per translation unit and are set with a stream-ordered copy,
// so the checks are exact for calls that are issued one after the other (what the tests do).  Launches that overlap
// on two streams (bload_epoch) register "anything" and are not checked.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include <initializer_list>

namespace bload {
namespace dbg {

enum KernelId { kNone = 0, kCopy = 7, kUnpackStaged = 8, kUnpackRagged = 9, kPackContig = 10, kCarry = 11, kResetState = 12,
                kRepeatLast = 14, kCopyVar = 16, kMetadata = 6, kTables = 5 };

// (the checker keeps one set of ranges per device: launches of a checked build never overlap each other)
#ifdef BLOAD_DEBUG
constexpr bool kChecked = true;
#else
constexpr bool kChecked = false;
#endif

#ifdef BLOAD_DEBUG
constexpr int kRanges = 6;
struct Ranges {
    const uint8_t* rd_lo[kRanges]; const uint8_t* rd_hi[kRanges];
    const uint8_t* wr_lo[kRanges]; const uint8_t* wr_hi[kRanges];
    int kernel;    // KernelId of the launch that follows; kNone = not checked
    int pad_;
};
static __device__ Ranges d_ranges;
// [0] accesses refused, [1] kernel id of the first, [2] 0 = read / 1 = write, [3] its address
static __device__ unsigned long long d_status[4];

__device__ __forceinline__ bool refuse(const void* p, int is_write)
{
    if (atomicAdd(&d_status[0], 1ULL) == 0) {
        d_status[1] = (unsigned long long)d_ranges.kernel;
        d_status[2] = (unsigned long long)is_write;
        d_status[3] = (unsigned long long)reinterpret_cast<uintptr_t>(p);
    }
    return false;
}
__device__ __forceinline__ bool may_read(const void* p, unsigned bytes)
{
    if (d_ranges.kernel == kNone) return true;
    const uint8_t* a = static_cast<const uint8_t*>(p);
#pragma unroll
    for (int i = 0; i < kRanges; ++i)
        if (a >= d_ranges.rd_lo[i] && a + bytes <= d_ranges.rd_hi[i]) return true;
    return refuse(p, 0);
}
__device__ __forceinline__ bool may_write(const void* p, unsigned bytes)
{
    if (d_ranges.kernel == kNone) return true;
    const uint8_t* a = static_cast<const uint8_t*>(p);
#pragma unroll
    for (int i = 0; i < kRanges; ++i)
        if (a >= d_ranges.wr_lo[i] && a + bytes <= d_ranges.wr_hi[i]) return true;
    return refuse(p, 1);
}

struct Span { const void* p; size_t bytes; };
// host: the ranges of the next launch on `st` (a null pointer or zero size is an empty range)
inline void expect(cudaStream_t st, int kernel, const Span (&reads)[kRanges], const Span (&writes)[kRanges])
{
    Ranges r;
    for (int i = 0; i < kRanges; ++i) {
        r.rd_lo[i] = static_cast<const uint8_t*>(reads[i].p); r.rd_hi[i] = r.rd_lo[i] + (reads[i].p ? reads[i].bytes : 0);
        r.wr_lo[i] = static_cast<const uint8_t*>(writes[i].p); r.wr_hi[i] = r.wr_lo[i] + (writes[i].p ? writes[i].bytes : 0);
    }
    r.kernel = kernel; r.pad_ = 0;
    (void)cudaMemcpyToSymbolAsync(d_ranges, &r, sizeof r, 0, cudaMemcpyHostToDevice, st);
}
inline void unchecked(cudaStream_t st)
{
    const Span none[kRanges] = {};
    expect(st, kNone, none, none);
}
// host: this translation unit's record, added to out[0] / copied to out[1..3] when it holds the first refusal seen
inline void collect(unsigned long long out[4], bool clear)
{
    unsigned long long s[4] = {0, 0, 0, 0};
    if (cudaMemcpyFromSymbol(s, d_status, sizeof s) != cudaSuccess) { (void)cudaGetLastError(); return; }
    if (s[0] && !out[0]) { out[1] = s[1]; out[2] = s[2]; out[3] = s[3]; }
    out[0] += s[0];
    if (clear) {
        const unsigned long long z[4] = {0, 0, 0, 0};
        (void)cudaMemcpyToSymbol(d_status, z, sizeof z);
    }
}
void register_collector(void (*fn)(unsigned long long[4], bool));
struct Registrar { Registrar() { register_collector(&collect); } };
static Registrar g_registrar;

#define BLOAD_MAY_READ(p, bytes) ::bload::dbg::may_read((p), (bytes))
#define BLOAD_MAY_WRITE(p, bytes) ::bload::dbg::may_write((p), (bytes))
#define BLOAD_DBG_EXPECT(st, kernel, ...) ::bload::dbg::expect_list((st), (kernel), __VA_ARGS__)
#define BLOAD_DBG_UNCHECKED(st) ::bload::dbg::unchecked(st)

// expect() with brace lists of up to kRanges spans: BLOAD_DBG_EXPECT(st, id, {{src, n}}, {{dst, m}})
struct SpanList {
    Span s[kRanges];
    SpanList(std::initializer_list<Span> l) : s{} { int i = 0; for (const Span& x : l) if (i < kRanges) s[i++] = x; }
};
inline void expect_list(cudaStream_t st, int kernel, SpanList reads, SpanList writes) { expect(st, kernel, reads.s, writes.s); }
#else
#define BLOAD_MAY_READ(p, bytes) true
#define BLOAD_MAY_WRITE(p, bytes) true
#define BLOAD_DBG_EXPECT(st, kernel, ...) ((void)0)
#define BLOAD_DBG_UNCHECKED(st) ((void)0)
#endif

}  // namespace dbg
}  // namespace bload

// Internal declarations shared by the translation units of libbload (GPU path only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bload.h"

namespace bload {

constexpr uint64_t kPlanMagic = 0x424c6f6164763031ULL;  // "BLoadv01"
constexpr size_t kAlign = 256;
constexpr int kHeaderBytes = 256;

// First 256 bytes of a plan buffer.
struct PlanHeader {
    uint64_t magic;
    int64_t n;
    int64_t n_blocks;
    int64_t sum_t;
    unsigned long long first_bad;  // ULLONG_MAX while no bad length was seen
    unsigned long long checksum;
    uint64_t seed;
    int32_t t_block;
    int32_t t_max;
    int32_t status;
    int32_t max_segs;
    uint32_t policy;
    uint32_t pad_[45];
};
static_assert(sizeof(PlanHeader) == kHeaderBytes, "header is 256 bytes");

// Device view of the tables of a plan (pointers resolved on the host from the offsets).
struct PlanView {
    PlanHeader* hdr;
    int64_t* offsets;
    int32_t* seg_seq;
    int32_t* seg_block;
    int32_t* seg_start;
    int64_t* seg_src;
    int32_t* block_seg_begin;
    int32_t* block_fill;
    int32_t* seq_block;
    int32_t* seq_start;
};

// Scratch layout of bload_plan.
struct WorkView {
    uint64_t* key_a;      // [n] sort keys (T << 32 | h), ping
    uint64_t* key_b;      // [n] pong
    int32_t* id_a;        // [n] payload ids, ping
    int32_t* id_b;        // [n] pong
    uint64_t* draw_u;     // [n] random word of draw k
    int4* draw_rec;       // [n] per draw: {length, unused count of that length before the draw, block, start}
    int64_t* partial;     // [chunks] per-chunk sums of lengths
    uint32_t* digit_hist; // [256 * (chunks + 1)] per-chunk digit counts of one sort pass, then the 256 digit totals
    int32_t* bucket_end;  // [t_block + 1] sequences with length <= l
};

// State of a fill rule that runs in several launches (bload_epoch): where the chain stands, and for every launch
// ("chunk") the blocks and draws it completed.  Lives in the scratch buffer, zeroed before the first chunk.
constexpr int kMaxEpochChunks = 32;
struct FillResume {
    int32_t k, b, room, start;               // next draw, open block, room left in it, its next free slot
    int32_t done, chunk;                     // all sequences placed; chunks run so far
    int32_t pad_[2];
    int32_t range[kMaxEpochChunks + 1][4];   // per chunk {first block, end block, end of the real blocks, 0}, clamped to
                                             // the caller's capacity; row kMaxEpochChunks: the filler blocks behind the plan
    int32_t draw[kMaxEpochChunks + 1][4];    // per chunk {first draw, end draw, first block, end block} (not clamped)
};
// Occupancy control of bload_epoch: the chunks of the fill rule ask for kChainSmemBytes of shared memory (they need
// far less) and every kernel that runs beside them asks for kBesideChainSmemBytes it never touches, so no CTA of
// those kernels fits on the SM that runs the chain (227 KB per SM), while three of them still fit on any other SM.
// A chain that shares its SM with copy warps was measured 30 % slower (its shared-memory loads queue behind their
// global loads and stores).
constexpr int kChainSmemBytes = 184 * 1024;
constexpr int kBesideChainSmemBytes = 46 * 1024;  // below the 48 KB a launch may ask for without opting in, static use included
struct EpochView {
    FillResume* resume;
    int32_t* fill_tables;  // snapshot of the fill rule's shared-memory tables between chunks
};
size_t epoch_layout(int32_t t_block, void* base, EpochView* v);

constexpr int kChunk = 2048;  // elements per CTA in scan / sort kernels (256 threads x 8)

inline size_t align_up(size_t x, size_t a = kAlign) { return (x + a - 1) / a * a; }
inline int64_t chunks_of(int64_t n) { return (n + kChunk - 1) / kChunk; }

size_t work_layout(int64_t n, int32_t t_block, void* base, WorkView* w);
void plan_layout(int64_t n, bload_sizes_t* s);
PlanView plan_view(void* d_plan, int64_t n);

// Extra scratch of the best-fit-decreasing planner (policy 2), placed after the WorkView region.
struct BfdView {
    int2* rec;            // [n] per item in placement order: {room it was taken from (0 = new block), room it left}
    uint64_t* ek_a;       // [n] event sort keys, ping
    uint64_t* ek_b;       // [n] pong
    int32_t* ei_a;        // [n] event payload (item index), ping
    int32_t* ei_b;        // [n] pong
    int32_t* put_item;    // [n] items ordered by (room they left, time)
    int32_t* jump_a;      // [n] predecessor pointers, ping
    int32_t* jump_b;      // [n] pong
    int32_t* blk;         // [n] block of item t
    int32_t* put_end;     // [t_block + 1] items that left a room <= r
    int32_t* take_end;    // [t_block + 1] items that took a room <= r (room 0 = opened a new block)
};
size_t bfd_layout(int64_t n, int32_t t_block, void* base, BfdView* v);

// stable LSD radix sort of (key, id) pairs on `digits` 8-bit digits starting at bit `first_shift`; the sorted
// arrays are returned in *k_out / *i_out (one of the two ping-pong pairs); and counts of keys by their high word
cudaError_t plan_radix_sort(uint64_t* ka, int32_t* ia, uint64_t* kb, int32_t* ib, int64_t n, int first_shift, int digits,
                            uint32_t* hist, const PlanHeader* hdr, cudaStream_t st, uint64_t** k_out, int32_t** i_out);
cudaError_t plan_key_buckets(const uint64_t* sorted_keys, int64_t n, int32_t max_value, int32_t* bucket_end,
                             const PlanHeader* hdr, cudaStream_t st);
cudaError_t launch_bfd(const PlanView& pv, const WorkView& wv, const BfdView& bv, const uint64_t* sorted_key,
                       const int32_t* sorted_id, int64_t n, int32_t t_block, cudaStream_t st);

// every kernel launch of the library goes through this counter (see bload_kernel_launches)
void count_launches(int k);

// which copy kernel a call chose (see bload_last_copy_kernel): 0 pack, 1 unpack, 2 carry_prev, 3 pack_var, 4 unpack_var
enum CopyCall { kCallPack = 0, kCallUnpack = 1, kCallCarryPrev = 2, kCallPackVar = 3, kCallUnpackVar = 4, kCopyCalls = 5 };
void note_copy_kernel(int call, const char* name);

unsigned int bulk_copy_timeouts();  // see bload_bulk_copy_timeouts

// Multiprocessors and shared memory per multiprocessor of the current device, asked for once per device (grids and
// occupancy are sized from them; a failed query answers with the B200's 148 and 228 KB).
struct DeviceInfo { int sm_count; int smem_per_sm; };
DeviceInfo device_info();
// cudaFuncAttributeMaxDynamicSharedMemorySize for `kernel` on the current device, set on the first call per device and
// kernel and remembered: the attribute call costs a few microseconds, which a per-batch launch would pay every time.
cudaError_t opt_in_shared_memory(const void* kernel, int bytes);
template <typename K>
inline cudaError_t opt_in_shared_memory(K* kernel, int bytes) { return opt_in_shared_memory(reinterpret_cast<const void*>(kernel), bytes); }

// launchers (each returns a cudaError_t from cudaPeekAtLastError)
cudaError_t launch_plan(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                        const PlanView& pv, const WorkView& wv, cudaStream_t st, cudaEvent_t* ev /*5 or null*/,
                        const BfdView* bv = nullptr /*policy 2 only*/);
// Programmatic dependent launch, used where one call issues two kernels that touch disjoint buffers (per-slot metadata,
// then the dense blocks): the first releases its dependents as soon as it runs, the second is launched with the
// programmatic-serialisation attribute and so starts beside it instead of behind it, and waits for it only at its own
// end, so that "the second has finished" still means "both have finished" for whatever comes next in the stream.
// Both instructions do nothing in a kernel that was launched the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void release_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void wait_for_prerequisites() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
#endif
cudaError_t launch_metadata(const PlanView& pv, int32_t t_block, int64_t block_begin, int64_t block_count,
                            int32_t* seq_id, int32_t* pos, uint8_t* reset, uint8_t* valid, cudaStream_t st,
                            const int32_t* d_range = nullptr, int64_t n = 0 /*sequences and frames of the plan, when the*/,
                            int64_t sum_t = 0 /*caller knows them: they choose the kernel*/);
cudaError_t launch_copy(bool unpack, const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                        int64_t block_count, const uint8_t* ragged_in, uint8_t* dense, uint8_t* ragged_out,
                        int64_t ragged_bytes, uint8_t pad_byte, cudaStream_t st, int64_t n, int64_t n_blocks,
                        bool gaps = false /*the plan's sequences do not tile the ragged buffer (chunks with deleted frames)*/,
                        bool beside_previous = false /*the launch before this one in `st` is the call's own metadata kernel,
                                                       which touches none of this launch's buffers: start beside it*/);
// The pieces of the planner and the copies that bload_epoch strings together on two streams.  `d_range` points to
// {first block, end block, end of the real blocks} in device memory: the blocks a launch covers are decided on the
// device, so these launches use fixed grids whose CTAs loop.
cudaError_t launch_plan_front(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                              const PlanView& pv, const WorkView& wv, cudaStream_t st, int32_t** sorted_id);
cudaError_t launch_fill_chunk(const PlanView& pv, const WorkView& wv, const EpochView& ev, int64_t n, int32_t t_block,
                              int32_t k_target, int32_t filler_end, cudaStream_t st);
cudaError_t launch_tables_chunk(const PlanView& pv, const WorkView& wv, const int32_t* sorted_id, int64_t n,
                                const int32_t* d_draw_range /*{first draw, end draw, first block, end block}*/,
                                cudaStream_t st);
cudaError_t launch_plan_finish(const PlanView& pv, cudaStream_t st);
cudaError_t launch_copy_range(bool unpack, const PlanView& pv, int32_t t_block, int64_t frame_bytes, const uint8_t* src,
                              uint8_t* dst, int64_t src_total_bytes, uint8_t pad_byte, const int32_t* d_range,
                              cudaStream_t st);

cudaError_t launch_var_offsets(const int32_t* lengths, const int32_t* rows, const int32_t* frame_bytes, int64_t n,
                               int64_t* out, int64_t* max_rows, cudaStream_t st);
cudaError_t launch_copy_var(bool unpack, const PlanView& pv, int32_t t_block, int32_t rows_max, int64_t row_stride,
                            int64_t block_begin, int64_t block_count, const int32_t* seq_rows, const int32_t* frame_bytes,
                            const int64_t* byte_offsets, const uint8_t* src, uint8_t* dst, uint8_t pad_byte, cudaStream_t st);
cudaError_t launch_carry_prev(const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                              int64_t block_count, const uint8_t* dense, uint8_t* prev, uint8_t fill_byte, cudaStream_t st,
                              int64_t n, int64_t sum_t);
bool staged_pack_with_metadata(const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                               int64_t block_count, const uint8_t* store, uint8_t* dense, int32_t* seq_id, int32_t* pos,
                               uint8_t* reset, uint8_t* valid, int64_t ragged_bytes, uint8_t pad_byte, cudaStream_t st,
                               int64_t n, cudaError_t* err);
cudaError_t launch_reset_state(const PlanView& pv, int64_t block_begin, int64_t block_count, int32_t slot, uint8_t* state,
                               int64_t state_bytes, const uint8_t* init, cudaStream_t st);
cudaError_t launch_repeat_last(const PlanView& pv, int32_t t_block, int64_t frame_bytes, int64_t block_begin,
                               int64_t block_count, uint8_t* dense, cudaStream_t st);
cudaError_t launch_valid_sum(const PlanView& pv, int32_t t_block, int64_t block_begin, int64_t block_count,
                             const float* values, double* block_sum, double* total, cudaStream_t st);

}  // namespace bload

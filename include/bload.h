/*
 * bload.h -- C ABI of libbload: BLoad's ragged-to-block packing on one NVIDIA B200 (sm_100a).
 *
 * The paper ("BLoad: Enhancing Neural Network Training with Efficient Sequential Data Handling",
 * section Methods) trains on N sequences of T_i frames without padding each to the longest one:
 * randomly sampled sequences are concatenated into blocks of a fixed number of frames, the tail
 * of a block that cannot be filled exactly is padded with zeros, and a table records the slot at
 * which each new sequence starts inside its block.  This library computes that assignment on the
 * GPU (bload_plan), materialises dense [blocks, t_block, frame] batches and their per-slot
 * metadata from a flat ragged frame store (bload_pack), scatters per-frame outputs back to the
 * ragged order (bload_unpack), and reports padding statistics (bload_stats).
 *
 * Conventions
 *   - "d_" pointers are DEVICE pointers; all others are HOST pointers.
 *   - The caller owns every buffer.  The library allocates no device memory and keeps no state
 *     between calls (apart from the benchmarking counters at the end of this file); a plan is
 *     position independent (tables addressed by byte offsets) and can
 *     be copied or saved as a blob of bload_sizes_t.plan_bytes bytes.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *   - Every function returns BLOAD_OK (0) or a negative BLOAD_ERR_* code.  Errors that the host
 *     can detect launch nothing.  Nothing aborts, throws or traps.
 *   - Frames are opaque byte strings of `frame_bytes` bytes; they are moved bit for bit.
 */
#ifndef BLOAD_H_
#define BLOAD_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define BLOAD_API __attribute__((visibility("default")))
#else
#define BLOAD_API
#endif

#define BLOAD_OK 0
#define BLOAD_ERR_NULL (-1)        /* a required pointer is NULL */
#define BLOAD_ERR_ARG (-2)         /* n < 1, t_block < 1, frame_bytes < 1, bad block range, ... */
#define BLOAD_ERR_LENGTH (-3)      /* some T_i outside [1, t_block]; index in info.first_bad_index */
#define BLOAD_ERR_WORKSPACE (-4)   /* plan or work buffer smaller than bload_plan_sizes says */
#define BLOAD_ERR_ALIGN (-5)       /* a device pointer is not aligned as documented */
#define BLOAD_ERR_UNSUPPORTED (-6) /* t_block above BLOAD_MAX_T_BLOCK, unknown policy */
#define BLOAD_ERR_CUDA (-7)        /* a CUDA runtime call or launch failed */
#define BLOAD_ERR_TIMEOUT (-8)     /* reserved: a bounded device-side wait expired.  No kernel of this version waits on a
                                      flag (the only waits are for the hardware's own copy groups), so no call returns it */
#define BLOAD_ERR_PLAN (-9)        /* info/plan do not describe a finished plan */

#define BLOAD_MAX_T_BLOCK 32768
#define BLOAD_POLICY_UNIFORM_SEQUENCES 0u /* every unused sequence that fits is equally likely */
#define BLOAD_POLICY_BEST_FIT_DECREASING 2u /* NOT the paper's rule: the textbook best-fit-decreasing heuristic, a
                                             deterministic low-padding comparison (seed only orders equal lengths) */
#define BLOAD_POLICY_CHUNKS_KEEP_TAIL 3u /* written into info.policy by bload_plan_chunks (not accepted by bload_plan) */
#define BLOAD_POLICY_CHUNKS_DROP_TAIL 4u
#define BLOAD_POLICY_UNIFORM_LENGTHS 1u   /* every length (key of L_dict) that fits and is not exhausted is equally
                                             likely, then the next unused sequence of that length; needs n < 2^26 */

/* Sizes and table offsets for a problem of n sequences (host only, no GPU call). */
typedef struct {
    size_t plan_bytes; /* bytes of the plan buffer */
    size_t work_bytes; /* bytes of the scratch buffer bload_plan needs (contents are garbage afterwards) */
    int64_t max_blocks; /* upper bound on n_blocks (= n); the tables below have room for it */
    /* byte offsets of the tables inside the plan buffer (each 256-byte aligned) */
    size_t off_offsets;         /* int64 [n+1]  first frame of sequence i in the ragged store; [n] = sum T */
    size_t off_seg_seq;         /* int32 [n]    sequence placed by the k-th draw (segments in placement order) */
    size_t off_seg_block;       /* int32 [n]    block of segment k */
    size_t off_seg_start;       /* int32 [n]    first slot of segment k in its block: the paper's start-index table */
    size_t off_seg_src;         /* int64 [n]    first frame of segment k in the ragged store (= offsets[seg_seq[k]]) */
    size_t off_block_seg_begin; /* int32 [max_blocks+1]  CSR: segments of block b are [begin[b], begin[b+1]) */
    size_t off_block_fill;      /* int32 [max_blocks]    occupied slots of block b; slots beyond are padding */
    size_t off_seq_block;       /* int32 [n]    inverse table: block of sequence i */
    size_t off_seq_start;       /* int32 [n]    inverse table: first slot of sequence i */
} bload_sizes_t;

/* Scalars of a finished plan (host). */
typedef struct {
    int32_t status;  /* BLOAD_OK or the error the planner found */
    int32_t t_block; /* block length in frames */
    int64_t n;       /* sequences */
    int64_t n_blocks;
    int64_t sum_t;   /* total frames */
    int64_t t_max;   /* longest sequence */
    int64_t first_bad_index; /* first i with T_i outside [1, t_block], else -1 */
    uint64_t checksum;       /* order-independent digest of (block, start, sequence) over all segments */
    int64_t max_segs_per_block;
    uint64_t seed;
    uint32_t policy;
    uint32_t n_source;       /* plans made by bload_plan_chunks: the sequences the chunks were cut from; else 0 */
} bload_plan_info_t;

typedef struct {
    int64_t n, sum_t, t_max, t_block, n_blocks;
    int64_t pad_packed;       /* n_blocks * t_block - sum_t */
    int64_t pad_naive_tmax;   /* n * t_max - sum_t  (every sample padded to the longest) */
    int64_t pad_naive_tblock; /* n * t_block - sum_t */
    int64_t min_blocks;       /* ceil(sum_t / t_block): no packing can use fewer blocks */
    double frac_packed;       /* pad_packed / (n_blocks * t_block) */
    double frac_naive_tmax;   /* pad_naive_tmax / (n * t_max) */
    double frac_naive_tblock;
    double reduction_vs_tmax; /* pad_naive_tmax / pad_packed (0 when pad_packed == 0) */
    double mean_segs_per_block;
    int64_t max_segs_per_block;
    int64_t frames_deleted;   /* 0 except for plans of bload_plan_chunks with BLOAD_CHUNKS_DROP_TAIL */
} bload_stats_t;

/*
 * bload_plan_sizes -- buffer sizes and table offsets for n sequences and blocks of t_block frames.
 * Host only.  Errors: NULL out, n < 1 or n >= 2^31, t_block < 1 (ARG), t_block > BLOAD_MAX_T_BLOCK
 * (UNSUPPORTED).
 */
BLOAD_API int bload_plan_sizes(int64_t n, int32_t t_block, bload_sizes_t* out);

/*
 * bload_plan -- block construction (paper, Methods, first paragraph; caption of the pseudocode
 * figure) and the table of start indices (Methods, second paragraph).
 *
 * Blocks are built one after another.  While some unused sequence is no longer than the room left
 * in the open block, one of them is drawn uniformly at random and appended (the paper's Random_*()
 * over L_dict); when none fits, the rest of the block is padding and the next block is opened.
 * Randomness comes from the counter-based generator Philox-4x64-10 keyed by `seed`, so the plan is
 * a pure function of (lengths, t_block, seed, policy).  `policy` selects the reading of "random entry"
 * (BLOAD_POLICY_UNIFORM_SEQUENCES, the default, or BLOAD_POLICY_UNIFORM_LENGTHS) or the deterministic
 * comparison strategy BLOAD_POLICY_BEST_FIT_DECREASING, which is not the paper's rule.
 *
 *   d_lengths  device int32[n], 4-byte aligned; every T_i must satisfy 1 <= T_i <= t_block
 *   d_plan     device buffer of plan_bytes bytes, 256-byte aligned; receives the tables
 *   d_work     device scratch of work_bytes bytes, 256-byte aligned
 *   info       host out; filled after ONE synchronisation of `stream` (the only one in the library)
 *
 * Returns info->status.  On BLOAD_ERR_LENGTH the tables are undefined and first_bad_index is set.
 */
BLOAD_API int bload_plan(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
               void* d_plan, size_t plan_bytes, void* d_work, size_t work_bytes, void* stream,
               bload_plan_info_t* info);

/*
 * bload_plan_async / bload_plan_finish -- bload_plan split in two, for callers that keep several plans
 * in flight.  The fill rule is a chain of dependent draws that occupies one warp of one SM, so plans
 * for different epochs (seeds) cost almost nothing extra when they run side by side on different
 * streams, and a plan for the next epoch can run under the pack/unpack traffic of the current one.
 *
 * bload_plan_async checks its arguments exactly like bload_plan, enqueues the planner on `stream` and
 * returns without synchronising (BLOAD_OK means "enqueued").  Each plan in flight needs its own d_plan
 * and d_work.  bload_plan_finish copies the plan's scalars to the host on `stream`, synchronises that
 * stream and fills `info` (all fields, taken from the plan itself); it returns info->status, and
 * BLOAD_ERR_PLAN if the buffer does not hold a finished plan.  The paper has no counterpart (it builds
 * its blocks on the host).
 */
BLOAD_API int bload_plan_async(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, uint32_t policy,
                               void* d_plan, size_t plan_bytes, void* d_work, size_t work_bytes, void* stream);
BLOAD_API int bload_plan_finish(const void* d_plan, void* stream, bload_plan_info_t* info);

/*
 * bload_epoch -- plan, metadata, pack and unpack of one whole epoch in a single call, with the copies running
 * while the plan is still being built.  Results are exactly those of
 *     bload_plan(policy BLOAD_POLICY_UNIFORM_SEQUENCES) ; bload_pack(blocks 0 .. block_capacity) ;
 *     bload_unpack(blocks 0 .. block_capacity)
 * but the fill rule (a chain of dependent draws that keeps one warp busy and leaves the memory system idle) runs
 * in chunks (about 1,800 draws each on average, at most 10, every chunk 1.25 times as long as the one before; or io->chunks
 * equal chunks) on `stream`, and as soon as a chunk has closed its blocks their tables, metadata,
 * pack and unpack are issued on `side_stream`, under the next chunk of the chain.  Only launch-order dependencies
 * (events) are used; no kernel waits for another.  The paper has no counterpart (it builds blocks on the host).
 *
 *   io->d_store / frame_bytes / d_dense      pack (skipped when d_dense is NULL)
 *   io->d_seq_id, d_pos, d_reset, d_valid    per-slot metadata, each may be NULL
 *   io->d_dense_out / out_frame_bytes / d_ragged_out   unpack (skipped when d_dense_out is NULL)
 *   io->block_capacity   rows (blocks) that d_dense, the metadata arrays and d_dense_out have; the number of
 *                        blocks is only known when the plan is done, so give an upper bound (the previous epoch's
 *                        count plus a margin, or 2 * sum_t / t_block + 1); rows beyond n_blocks are filler
 *   d_work / work_bytes  as for bload_plan (bload_plan_sizes covers this call)
 *   side_stream          a second stream of the same device, or NULL (then everything runs on `stream`, in order);
 *                        give `stream` the higher priority of the two, so that each chunk of the chain starts as
 *                        soon as an SM has room for it
 *
 * Both streams are synchronised once before the call returns: on return `info` is filled and every output is
 * complete.  Errors are those of bload_plan, bload_pack and bload_unpack; BLOAD_ERR_WORKSPACE is also returned when
 * n_blocks exceeds block_capacity (the plan is complete and info->n_blocks tells how many rows are needed; blocks
 * beyond the capacity were not packed).  With bload_set_plan_timing(1), bload_epoch_stage_times returns the device
 * time of the last call, summed over chunks: [0] fill rule, [1] tables, [2] metadata, [3] pack, [4] unpack (ms).
 */
typedef struct {
    const void* d_store;
    int64_t frame_bytes;
    void* d_dense;
    int32_t* d_seq_id;
    int32_t* d_pos;
    uint8_t* d_reset;
    uint8_t* d_valid;
    const void* d_dense_out;
    int64_t out_frame_bytes;
    void* d_ragged_out;
    int64_t block_capacity;
    uint8_t pad_byte;
    uint8_t chunks;      /* launches of the fill rule: 0 = chosen by the library, else 1..32 */
    uint8_t reserved_[6];
} bload_epoch_io_t;
BLOAD_API int bload_epoch(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed, void* d_plan,
                          size_t plan_bytes, void* d_work, size_t work_bytes, const bload_epoch_io_t* io, void* stream,
                          void* side_stream, bload_plan_info_t* info);
BLOAD_API int bload_epoch_stage_times(float out_ms[5]);

/*
 * bload_pack -- dense batches and per-slot metadata for blocks [block_begin, block_begin+block_count)
 * (paper, Methods: concatenate the sequences of a block, pad the rest with zeros; the start table).
 *
 *   d_dense[q, s, :] = d_store[(offsets[id] + f) * frame_bytes ...]  if slot s of block block_begin+q
 *                      holds frame f of sequence id;  pad_byte repeated frame_bytes times otherwise
 *   d_seq_id[q, s] = id or -1     d_pos[q, s] = f or -1
 *   d_reset[q, s]  = 1 at the first slot of every sequence, else 0 (where carried state must be reset)
 *   d_valid[q, s]  = 1 on frames, 0 on padding
 *
 * Blocks at or beyond n_blocks are filler (all padding, all flags 0, ids -1) so that a caller can
 * round an epoch up to whole batches.  d_store is the flat ragged store (sum_t * frame_bytes bytes,
 * sequence i at frame offsets[i]); d_dense is [block_count, t_block, frame_bytes] row major.
 * d_store and d_dense must be 16-byte aligned.  d_dense and each of the four metadata outputs may be
 * NULL (that output is skipped).  Asynchronous on `stream`; no host synchronisation.  Launches: one kernel for the
 * metadata and one for the dense blocks; a call that asks for both, for small word-sized frames (frame_bytes a multiple
 * of 4, runs of at most 16 KB on average, blocks of less than 1 GiB) and at most 4 Mi slots, is a single
 * launch -- the call a training loop makes per batch of token-sized frames is bound by launch overhead, not by bytes.
 * With large frames the two kernels run side by side (the second is a programmatic dependent launch that does not wait
 * for the first to end: their outputs are disjoint); whatever follows in `stream` still starts after both have ended.
 * So the dense buffer and the metadata arrays of one call must not overlap each other.
 * Errors: NULL plan/info/store (when d_dense is given), ARG (frame_bytes < 1, negative range,
 * block_begin + block_count >= 2^31), ALIGN, PLAN (info->status != 0), CUDA.
 */
BLOAD_API int bload_pack(const void* d_plan, const bload_plan_info_t* info, const void* d_store, int64_t frame_bytes,
               int64_t block_begin, int64_t block_count, void* d_dense, int32_t* d_seq_id, int32_t* d_pos,
               uint8_t* d_reset, uint8_t* d_valid, uint8_t pad_byte, void* stream);

/*
 * bload_pack_repeat_last -- bload_pack with the other padding the paper mentions (caption of its figure
 * of the naive padding solution: samples are padded "by adding 0's or repeating the last entry"): the
 * padding slots of a block repeat the frame in the block's last occupied slot instead of holding
 * pad_byte.  Filler blocks, which hold no frame, are still filled with pad_byte, and the metadata is
 * that of bload_pack (padding stays valid = 0: the repeated frames are not data).  Same arguments,
 * alignment rules and errors as bload_pack.  Runs the pack kernels and then one small kernel that
 * rewrites the padding from the dense buffer itself, on the same stream.
 */
BLOAD_API int bload_pack_repeat_last(const void* d_plan, const bload_plan_info_t* info, const void* d_store,
                                     int64_t frame_bytes, int64_t block_begin, int64_t block_count, void* d_dense,
                                     int32_t* d_seq_id, int32_t* d_pos, uint8_t* d_reset, uint8_t* d_valid,
                                     uint8_t pad_byte, void* stream);

/*
 * bload_unpack -- inverse of bload_pack for per-frame outputs: for every valid slot of the given
 * blocks, d_ragged_out[(offsets[id] + f) * out_frame_bytes ...] = d_dense_out[q, s, :].  Padding
 * slots and filler blocks are ignored; frames of sequences outside the block range are not touched.
 * The paper does not describe this step; it is defined as the exact inverse of the gather above.
 * Both buffers 16-byte aligned.  Asynchronous on `stream`.
 */
BLOAD_API int bload_unpack(const void* d_plan, const bload_plan_info_t* info, const void* d_dense_out,
                 int64_t out_frame_bytes, int64_t block_begin, int64_t block_count, void* d_ragged_out,
                 void* stream);

/*
 * Frames whose size differs from sample to sample (paper, Problem Statement: each sample S_i has its
 * own H, W and T).  Sequence i holds T_i frames of F_i = d_frame_bytes[i] bytes, back to back, at byte
 * d_byte_offsets[i] of the store.  A slot of a block has slot_bytes bytes (at least the largest F_i);
 * a frame sits at the start of its slot and the rest of the slot is padding.  The plan is the ordinary
 * one (it depends only on the lengths), and per-slot metadata comes from bload_pack as before.  The
 * paper does not say how frames of different sizes share a block; this layout (every frame on a
 * canvas of the largest size, as opaque bytes) is the reading taken here.
 *
 * bload_var_offsets -- d_byte_offsets[i] = sum over j < i of T_j * F_j, for i = 0..n.  The array needs
 * n + 3 elements: [n] = total bytes of the store, [n+1] = largest F_i, [n+2] = first i with F_i < 1
 * or -1; the same three values are returned in `info` after one synchronisation of `stream`.
 * Returns BLOAD_ERR_ARG when some F_i < 1.  d_lengths, d_frame_bytes: device int32[n].
 *
 * bload_pack_var / bload_unpack_var -- bload_pack / bload_unpack with per-sequence frame sizes:
 *   d_dense[q, s, 0:F_id] = frame f of sequence id;  d_dense[q, s, F_id:slot_bytes] = pad_byte
 *   d_ragged_out[byte_offsets[id] + f * F_id ...] = d_dense_out[q, s, 0:F_id]
 * d_dense is [block_count, t_block, slot_bytes]; store, dense and ragged_out 16-byte aligned.
 * Precondition: 1 <= F_i <= slot_bytes for every i (bload_var_offsets reports the largest); sizes
 * outside that range are clamped on the device, which truncates frames but never leaves the buffers.
 * Asynchronous on `stream`.  Errors as for bload_pack (slot_bytes in the place of frame_bytes).
 */
typedef struct {
    int64_t total_bytes;     /* bytes of the ragged store */
    int64_t max_frame_bytes; /* largest F_i: the smallest slot_bytes that holds every frame */
    int64_t first_bad_index; /* first i with F_i < 1 (or rows_i < 1), else -1 */
    int64_t max_rows;        /* most rows of any image (1 for the calls without rows) */
} bload_var_info_t;
BLOAD_API int bload_var_offsets(const int32_t* d_lengths, const int32_t* d_frame_bytes, int64_t n,
                                int64_t* d_byte_offsets, void* stream, bload_var_info_t* info);
BLOAD_API int bload_pack_var(const void* d_plan, const bload_plan_info_t* info, const void* d_store,
                             const int32_t* d_frame_bytes, const int64_t* d_byte_offsets, int64_t slot_bytes,
                             int64_t block_begin, int64_t block_count, void* d_dense, uint8_t pad_byte, void* stream);
BLOAD_API int bload_unpack_var(const void* d_plan, const bload_plan_info_t* info, const void* d_dense_out,
                               const int32_t* d_frame_bytes, const int64_t* d_byte_offsets, int64_t slot_bytes,
                               int64_t block_begin, int64_t block_count, void* d_ragged_out, void* stream);

/*
 * The same with frames as images (the H x W of the paper's problem statement): every frame of sequence i has
 * d_rows[i] rows of d_row_bytes[i] bytes (row major, rows back to back in the store).  A slot is a canvas of
 * rows_max rows of row_stride bytes, so d_dense is [block_count, t_block, rows_max, row_stride]; an image sits in
 * the top left corner of its canvas, and the bytes to its right and below it are pad_byte.  With one row per image
 * and rows_max == 1 these calls are bload_pack_var / bload_unpack_var.
 *
 * bload_var_offsets2d -- d_byte_offsets[i] = sum over j < i of T_j * rows_j * row_bytes_j.  The array needs n + 4
 * elements: [n] total bytes, [n+1] largest row size, [n+2] first i with a size < 1 or -1, [n+3] most rows; the same
 * values come back in `info`.  Precondition of the pack / unpack calls: 1 <= rows_i <= rows_max and
 * 1 <= row_bytes_i <= row_stride (clamped on the device otherwise, as above).  Errors as for the calls above.
 */
BLOAD_API int bload_var_offsets2d(const int32_t* d_lengths, const int32_t* d_rows, const int32_t* d_row_bytes, int64_t n,
                                  int64_t* d_byte_offsets, void* stream, bload_var_info_t* info);
BLOAD_API int bload_pack_var2d(const void* d_plan, const bload_plan_info_t* info, const void* d_store,
                               const int32_t* d_rows, const int32_t* d_row_bytes, const int64_t* d_byte_offsets,
                               int64_t rows_max, int64_t row_stride, int64_t block_begin, int64_t block_count,
                               void* d_dense, uint8_t pad_byte, void* stream);
BLOAD_API int bload_unpack_var2d(const void* d_plan, const bload_plan_info_t* info, const void* d_dense_out,
                                 const int32_t* d_rows, const int32_t* d_row_bytes, const int64_t* d_byte_offsets,
                                 int64_t rows_max, int64_t row_stride, int64_t block_begin, int64_t block_count,
                                 void* d_ragged_out, void* stream);

/*
 * Consumer side of the start table (paper, Methods, second paragraph, and its figure of the DDS
 * architecture): a recurrent model feeds information of frame t-1 into frame t, and the table of
 * start indices tells it where that information belongs to another sequence and has to be
 * discarded.  The three calls below apply the table on the GPU, straight from the plan.
 *
 * bload_carry_prev -- what every slot receives from the slot before it, for a whole batch at once:
 *
 *   d_prev[q, s, :] = d_dense[q, s-1, :]   if slot s of block block_begin+q holds frame f >= 1 of a
 *                                          sequence (slot s-1 then holds frame f-1 of the same one)
 *                   = fill_byte repeated   on the first frame of every sequence, on padding and in
 *                                          filler blocks (nothing is carried over there)
 *
 * d_dense and d_prev are [block_count, t_block, frame_bytes] row major, 16-byte aligned, and must
 * not be the same buffer (ARG) nor overlap.  Frames are opaque bytes.  Asynchronous on `stream`.
 * Errors as for bload_pack.
 */
BLOAD_API int bload_carry_prev(const void* d_plan, const bload_plan_info_t* info, const void* d_dense,
                               int64_t frame_bytes, int64_t block_begin, int64_t block_count, void* d_prev,
                               uint8_t fill_byte, void* stream);

/*
 * bload_reset_state -- one step of a recurrence that walks the slots of a batch in order.  Call it
 * before slot `slot` is processed: row q of the carried state (d_state, [block_count, state_bytes]
 * row major, opaque bytes) is overwritten with the initial state unless a sequence continues at that
 * slot of block block_begin+q, that is, on the first frame of a sequence, on padding and in filler
 * blocks.  Rows whose sequence continues are not touched.  d_init points to state_bytes bytes of
 * initial state (device, 16-byte aligned) or is NULL for zeros.  Asynchronous on `stream`.
 * Errors: NULL plan/info/state, ARG (state_bytes < 1, slot outside [0, t_block), bad range), ALIGN,
 * PLAN, CUDA.
 */
BLOAD_API int bload_reset_state(const void* d_plan, const bload_plan_info_t* info, int64_t block_begin,
                                int64_t block_count, int32_t slot, void* d_state, int64_t state_bytes,
                                const void* d_init, void* stream);

/*
 * bload_valid_sum -- masked reduction of per-slot values (a per-frame loss, say): padding slots and
 * filler blocks hold no frame and must not count.
 *
 *   d_block_sum[q] = sum over the frames s of block block_begin+q of d_values[q, s]      (double)
 *   d_total[0]     = sum over q of d_block_sum[q];  d_total[1] = number of frames in the range
 *
 * d_values is float32 [block_count, t_block] (4-byte aligned; 16-byte aligned rows are read as
 * vectors); d_block_sum is double[block_count]; d_total is double[2] or NULL (skipped).  Sums are
 * accumulated in double precision in a fixed order, so repeated calls give identical bits; against a
 * sum taken in another order the difference is bounded by block rounding, about 1e-15 of the sum of
 * magnitudes.  A mean over frames is d_total[0] / d_total[1].  Asynchronous on `stream`.
 * Errors: NULL plan/info/values/block_sum, ARG (bad range), ALIGN, PLAN, CUDA.
 */
BLOAD_API int bload_valid_sum(const void* d_plan, const bload_plan_info_t* info, const float* d_values,
                              int64_t block_begin, int64_t block_count, double* d_block_sum, double* d_total,
                              void* stream);

/*
 * bload_stats -- padding statistics from the scalars of a plan (host only; closed forms).
 * pad_naive_tmax is the "0 padding" row of the paper's Table I, pad_packed its "block_pad" row.
 * For a plan of bload_plan_chunks the samples are the chunks: n = n_chunks = n_blocks, t_max = longest chunk,
 * pad_packed = n_chunks * t_chunk - frames kept, frames_deleted = frames of the store - frames kept, and the
 * naive-padding fields describe padding every chunk to the longest chunk.
 */
BLOAD_API int bload_stats(const bload_plan_info_t* info, bload_stats_t* out);

/*
 * The chunking strategy that the paper compares BLoad with (section "Problem Statement and Current Limitations":
 * every sample is broken into chunks of T_block frames and every chunk is treated as an individual sample; figure
 * "Sampling solution"; Table I, column "sampling").  Built as a planner only, so that its padding and deleted frames
 * can be put beside BLoad's on the same data and its batches come out of the same kernels.
 *
 * Sequence i (any T_i >= 1; it may be longer than t_chunk) is cut at frames 0, t_chunk, 2 t_chunk, ...
 *   BLOAD_CHUNKS_KEEP_TAIL  the last, shorter chunk is kept and padded: nothing is deleted
 *   BLOAD_CHUNKS_DROP_TAIL  only full chunks are kept: no padding, the last T_i mod t_chunk frames of every sequence
 *                           are deleted (the reading under which the table's "sampling" column has zero padding and
 *                           a count of deleted frames)
 * Chunks are numbered in order of (sequence, position).  The plan that bload_plan_chunks writes is an ordinary plan
 * of n_chunks "sequences" in blocks of t_chunk slots: chunk j is sequence j, alone in block j from slot 0, and its
 * entry of the offsets table is its first frame in the ORIGINAL ragged store ([n_chunks] = all frames of that store),
 * so bload_pack, bload_unpack (deleted frames are never touched), bload_carry_prev, bload_reset_state,
 * bload_valid_sum and bload_stats take it as it is.  Per-slot metadata then names chunks: seq_id = chunk number,
 * pos = position inside the chunk, reset = 1 at slot 0 of every block -- which is the strategy's weakness the paper
 * points out: state cannot be carried from one chunk of a sequence to the next.  d_chunk_seq / d_chunk_first
 * (int32[n_chunks], each may be NULL) receive the sequence each chunk was cut from and its first frame there.
 * The calls for per-sequence frame sizes (bload_pack_var ...) do not accept such a plan (BLOAD_ERR_UNSUPPORTED).
 *
 * bload_chunk_count   the totals, after one synchronisation of `stream`; needs them before the plan can be sized
 * bload_plan_chunks   the plan; n_chunks as counted (BLOAD_ERR_ARG if the lengths give another number); plan_bytes at
 *                     least bload_plan_sizes(n_chunks, t_chunk).plan_bytes; one synchronisation of `stream`
 * d_work: device scratch of bload_chunk_work_bytes(n) bytes, 256-byte aligned (both calls).
 * Errors: NULL, ARG (n < 1, t_chunk < 1, unknown tail, n_chunks < 1: with DROP_TAIL every sequence may be shorter
 * than a chunk, then there is nothing to plan), UNSUPPORTED (t_chunk > BLOAD_MAX_T_BLOCK), LENGTH (some T_i < 1, index
 * in first_bad_index), WORKSPACE, ALIGN, CUDA.
 */
#define BLOAD_CHUNKS_KEEP_TAIL 0u
#define BLOAD_CHUNKS_DROP_TAIL 1u
typedef struct {
    int32_t status;
    uint32_t tail;
    int32_t t_chunk;
    int32_t reserved_;
    int64_t n;               /* sequences */
    int64_t n_chunks;        /* = blocks */
    int64_t frames_kept;
    int64_t frames_deleted;  /* Table I, row "# frames deleted" */
    int64_t pad_frames;      /* Table I, row "padding amount": n_chunks * t_chunk - frames_kept */
    int64_t sum_t;           /* frames of the ragged store */
    int64_t t_max;           /* longest sequence */
    int64_t first_bad_index; /* first i with T_i < 1, else -1 */
} bload_chunk_info_t;
BLOAD_API size_t bload_chunk_work_bytes(int64_t n);
BLOAD_API int bload_chunk_count(const int32_t* d_lengths, int64_t n, int32_t t_chunk, uint32_t tail, void* d_work,
                                size_t work_bytes, void* stream, bload_chunk_info_t* out);
BLOAD_API int bload_plan_chunks(const int32_t* d_lengths, int64_t n, int32_t t_chunk, uint32_t tail, int64_t n_chunks,
                                void* d_plan, size_t plan_bytes, void* d_work, size_t work_bytes, int32_t* d_chunk_seq,
                                int32_t* d_chunk_first, void* stream, bload_plan_info_t* info);

/*
 * bload_plan_static -- bload_plan for callers that must not, or cannot, allocate device memory.
 * (The paper has no counterpart of this call; it is a packaging variant of bload_plan and computes
 * exactly the same plan.)
 *
 * bload_plan needs a scratch buffer from its caller.  A data-loading thread that lives next to a
 * training job usually cannot get one: the framework's caching allocator has already taken the
 * device's memory, so a new cudaMalloc may fail, and even when it succeeds it can stall every
 * stream on the device while the driver serves it.  The same goes for loops that are simply
 * forbidden to touch the allocator.  This entry point keeps its scratch in a fixed array of
 * BLOAD_STATIC_SCRATCH_BYTES bytes inside the library image, so it calls no cudaMalloc, no
 * cudaFree and no allocating routine of any library.  The price: every GPU that loads the
 * library holds those bytes until the process exits, and the problem size is capped.
 *
 *   d_lengths, n, t_block, seed, d_plan, plan_bytes, stream, info: as for bload_plan
 *   (the caller still provides the input and the plan buffer; only d_work/work_bytes are gone).
 *   policy: BLOAD_POLICY_UNIFORM_SEQUENCES or BLOAD_POLICY_UNIFORM_LENGTHS, the two readings of the
 *   paper's rule.  BLOAD_POLICY_BEST_FIT_DECREASING needs more scratch per sequence than the array
 *   was sized for and returns BLOAD_ERR_UNSUPPORTED here; use bload_plan for it.
 *
 * Limits and errors: n > BLOAD_STATIC_MAX_N, or a (n, t_block) whose scratch need exceeds the
 * array, returns BLOAD_ERR_WORKSPACE ("buffer too small") and launches nothing; use bload_plan
 * with your own buffer for larger problems.  All other errors are those of bload_plan.
 *
 * First call on a device: the library looks up the device address of its array (the current
 * device must be the one the buffers live on).  Make that first call outside any stream capture.
 *
 * Sharing: all calls on a device use the same array and it keeps whatever the last call left.
 * The planner overwrites every scratch table it reads, so nothing has to be cleared between
 * calls; but two calls whose kernels overlap on the GPU (different streams or threads) race on
 * the array and produce garbage.  Run them one after the other, as this call itself does: like
 * bload_plan it synchronises `stream` once before it returns.
 */
#define BLOAD_STATIC_MAX_N 65536
#define BLOAD_STATIC_SCRATCH_BYTES (4u << 20)
BLOAD_API int bload_plan_static(const int32_t* d_lengths, int64_t n, int32_t t_block, uint64_t seed,
                                uint32_t policy, void* d_plan, size_t plan_bytes, void* stream,
                                bload_plan_info_t* info);

/*
 * bload_rank_range -- the share of one data-parallel rank, host only.
 *
 * The paper's motivation (section "Problem Statement and Current Limitations"): with data-parallel
 * training every process must run the same number of equally long iterations, or gradient
 * synchronisation stalls without an error.  Blocks all have t_block slots, so it is enough to give
 * every rank the same number of blocks: ranks take contiguous ranges of `per_rank` blocks, where
 * per_rank is ceil(n_blocks / world_size) rounded up to a whole number of batches of `batch_blocks`.
 * Ranges may reach beyond n_blocks; bload_pack writes such blocks as padding (filler) and
 * bload_unpack ignores them, so every rank can run the same loop.  No communication is involved:
 * each rank computes the same plan from the same seed and packs only its range.
 *
 * out_begin / out_count receive the rank's first block and its number of blocks (equal for all ranks).
 * Errors: NULL outputs, n_blocks < 1, world_size < 1, rank outside [0, world_size), batch_blocks < 1,
 * or a range that would not fit a 31-bit block index (BLOAD_ERR_ARG).
 */
BLOAD_API int bload_rank_range(int64_t n_blocks, int32_t world_size, int32_t rank, int32_t batch_blocks,
                               int64_t* out_begin, int64_t* out_count);

/*
 * bload_plan_stage_times -- device time, in milliseconds, that the most recent bload_plan call of
 * this thread spent in each stage: [0] validate + scan + keys, [1] key sort, [2] fill rule,
 * [3] inverse tables.  Host only; for benchmarking.  Returns BLOAD_ERR_PLAN when no plan was timed.
 * Timing is enabled by bload_set_plan_timing(1) (off by default).  It creates, records and destroys five
 * events per plan; on the test machine that was enough to keep host<->device copies on other streams from
 * overlapping, so switch it on only around the plans whose stages are to be timed.
 */
BLOAD_API int bload_set_plan_timing(int enable);
BLOAD_API int bload_plan_stage_times(float out_ms[4]);

/*
 * bload_kernel_launches -- number of kernels this library has launched in this process so far
 * (all threads).  Host only; lets a benchmark report how many launches a timed region contained.
 */
BLOAD_API int64_t bload_kernel_launches(void);

/*
 * bload_debug_status -- what the bounds-checking build of the library has seen.  That build (compiled with
 * -DBLOAD_DEBUG as libbload_debug.so) checks every global-memory access of its copy, metadata and table kernels
 * against the buffer ranges of the call, skips an access that lies outside them and records it; nothing traps.
 * out[0] = accesses refused since the last clear, out[1] = number of the kernel with the first one (5 tables,
 * 6 metadata, 7 to 11 and 16 the copy kernels, 12 state reset, 14 repeat-last), out[2] = 0 read / 1 write,
 * out[3] = its address.  Synchronises the device.  `clear` != 0 resets the record.  The ordinary build returns
 * BLOAD_ERR_UNSUPPORTED and zeros.  Calls that run kernels on two streams at once (bload_epoch) are not checked.
 */
BLOAD_API int bload_debug_status(uint64_t out[4], int clear);

/*
 * bload_last_copy_kernel -- name of the copy kernel that the most recent call of this host thread launched for
 * which = 0 bload_pack (the dense output), 1 bload_unpack, 2 bload_carry_prev, 3 bload_pack_var[2d],
 * 4 bload_unpack_var[2d].  The library picks a kernel from the frame size and the run lengths (register path for
 * large frames, shared-memory staged paths for small word-sized frames, run by run or -- for short runs -- word by
 * word, unstaged walks word by word or, for frames of 1 to 3 bytes, in granules of 16 bytes); a benchmark reports the
 * choice with this
 * call instead of guessing it.  Host only.  Returns "" when no such call was made, or for another `which`.
 */
BLOAD_API const char* bload_last_copy_kernel(int which);

/*
 * bload_bulk_copy_timeouts -- for builds with -DBLOAD_BULK_COPY=1 only (a measurement variant that sends large frames
 * through the bulk-copy engine and waits on mbarriers; the default library has no such wait and returns 0): the number
 * of mbarrier waits that gave up after their poll limit since the library was loaded.  A warp that gives up stops
 * copying, so any value but 0 means incomplete outputs.  Synchronises the device.  Host only.
 */
BLOAD_API int64_t bload_bulk_copy_timeouts(void);

BLOAD_API const char* bload_strerror(int code);
BLOAD_API int bload_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BLOAD_H_ */

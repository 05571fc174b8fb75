/*
 * bload_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, single-threaded CPU statement of BLoad's ragged-to-block
 * packing (Methods section of the paper, its Fig. "Our proposed padding
 * approach" and the caption of its pseudocode figure).  It exists so that the
 * GPU library can be compared with it element by element.  It shares no code
 * with the GPU library and must never be called from the product path: only
 * the tests, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * Everything is written with linear scans, per-slot loops and memcpy so that a
 * reader can check each function against the paper by eye.
 *
 * Pins (what each function is checked against, in tests that need no GPU):
 *   philox4x64_10      numpy's Philox bit generator (same published algorithm)
 *   oracle_pick        Python big-integer arithmetic
 *   offsets            numpy.cumsum (textbook exclusive prefix sum)
 *   L_dict order       Python sorted() on (T, h, i)
 *   fill rule          exhaustive enumeration of the choice tree on tiny inputs
 *                      (reachable set, exact probabilities, chi-square),
 *                      maximality and no-drop/no-split invariants, the toy
 *                      dataset of the paper (8 videos, lengths 2..6)
 *   plan digest        recomputed from the segment list with Python integers (MurmurHash3's
 *                      published finaliser typed in the test), on plans whose block and
 *                      sequence numbers pass 2^16; field swaps and reorderings
 *   stats              closed forms; the paper's Table I "0 padding" count
 *   metadata/pack/unpack  numpy fancy-index gather built from the tables,
 *                      round trip, pad bytes
 *   pack_repeat_last   numpy gather with pad slots mapped to the block's last frame; with one
 *                      sequence per block, the paper's naive repeat-last padding of each sample
 *   byte_offsets       numpy.cumsum of T_i * F_i
 *   pack_var/unpack_var  equal frame sizes reduce to pack/unpack; per-slot numpy construction from
 *                      H_i x W_i images; round trip; padding bytes
 *   pack_var2d/unpack_var2d  numpy canvases (canvas[:H_i, :W_i] = image); one row per image reduces to
 *                      pack_var; round trip
 *   carry_prev         shifting every sequence by one frame in the ragged store and
 *                      packing that gives the same bytes
 *   reset_state        a running sum carried through the slots with resets equals the
 *                      per-sequence numpy.cumsum after unpacking
 *   valid_sum          packing per-frame integers and summing the frames equals the sum
 *                      over the ragged array (exact in double)
 *   chunks             closed forms with numpy (sum of ceil / floor of T_i / c, T_i mod c), every kept frame
 *                      in exactly one chunk, chunks of one sequence in order; a chunk length that
 *                      covers every sequence reduces to the paper's naive padding (Table I,
 *                      "0 padding" = 534831); chunk pack/unpack/metadata against the ordinary
 *                      functions run on the derived one-chunk-per-block plan, and against numpy
 *   Parity unpinned: the paper's "block_pad" padding count of Table I (block
 *   length of that run is not stated and the rule is random) and its
 *   time-per-epoch figures.
 */
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_ERR_ARG (-1)
#define ORACLE_ERR_LENGTH (-2)
#define ORACLE_ERR_NOMEM (-3)
#define ORACLE_ERR_POLICY (-4)

/* ------------------------------------------------------------------------ */
/* Counter-based random numbers: Philox-4x64-10 (Salmon, Moraes, Dror, Shaw, */
/* "Parallel random numbers: as easy as 1, 2, 3", SC'11).                    */
/* ------------------------------------------------------------------------ */

static void mul_hi_lo(uint64_t a, uint64_t b, uint64_t *hi, uint64_t *lo)
{
    unsigned __int128 p = (unsigned __int128)a * (unsigned __int128)b;
    *hi = (uint64_t)(p >> 64);
    *lo = (uint64_t)p;
}

void oracle_philox4x64_10(const uint64_t ctr_in[4], const uint64_t key_in[2], uint64_t out[4])
{
    const uint64_t mult0 = 0xD2E7470EE14C6C93ULL, mult1 = 0xCA5A826395121157ULL;
    const uint64_t weyl0 = 0x9E3779B97F4A7C15ULL, weyl1 = 0xBB67AE8584CAA73BULL;
    uint64_t c[4] = {ctr_in[0], ctr_in[1], ctr_in[2], ctr_in[3]};
    uint64_t k[2] = {key_in[0], key_in[1]};
    for (int round = 0; round < 10; ++round) {
        uint64_t hi0, lo0, hi1, lo1;
        if (round > 0) { k[0] += weyl0; k[1] += weyl1; }
        mul_hi_lo(mult0, c[0], &hi0, &lo0);
        mul_hi_lo(mult1, c[2], &hi1, &lo1);
        uint64_t n0 = hi1 ^ c[1] ^ k[0];
        uint64_t n1 = lo1;
        uint64_t n2 = hi0 ^ c[3] ^ k[1];
        uint64_t n3 = lo0;
        c[0] = n0; c[1] = n1; c[2] = n2; c[3] = n3;
    }
    out[0] = c[0]; out[1] = c[1]; out[2] = c[2]; out[3] = c[3];
}

/* Two streams of the generator: key = (seed, stream), counter = (index,0,0,0),
 * first output word is used. */
#define STREAM_KEYS 1ULL
#define STREAM_DRAWS 2ULL

/* h_i: the shuffle key that orders sequences of equal length inside L_dict. */
uint32_t oracle_seq_key(uint64_t seed, int64_t i)
{
    uint64_t c[4] = {(uint64_t)i, 0, 0, 0}, k[2] = {seed, STREAM_KEYS}, o[4];
    oracle_philox4x64_10(c, k, o);
    return (uint32_t)(o[0] >> 32);
}

/* u_k: the 64-bit random word of the k-th draw of the fill loop. */
uint64_t oracle_draw_word(uint64_t seed, int64_t k)
{
    uint64_t c[4] = {(uint64_t)k, 0, 0, 0}, kk[2] = {seed, STREAM_DRAWS}, o[4];
    oracle_philox4x64_10(c, kk, o);
    return o[0];
}

/* Map a 64-bit word to an index in [0, m): floor(u * m / 2^64). */
uint64_t oracle_pick(uint64_t u, uint64_t m)
{
    return (uint64_t)(((unsigned __int128)u * (unsigned __int128)m) >> 64);
}

/* ------------------------------------------------------------------------ */
/* Ragged offsets: offsets[i] = T_0 + ... + T_{i-1}; offsets[n] = sum T.     */
/* (Problem statement: N samples of T_i frames stored back to back.)         */
/* ------------------------------------------------------------------------ */
void oracle_offsets(const int32_t *lengths, int64_t n, int64_t *offsets)
{
    int64_t acc = 0;
    for (int64_t i = 0; i < n; ++i) { offsets[i] = acc; acc += lengths[i]; }
    offsets[n] = acc;
}

/* ------------------------------------------------------------------------ */
/* Plan: block construction (Methods, first paragraph) and the table of      */
/* start indices (Methods, second paragraph).                                */
/* ------------------------------------------------------------------------ */
typedef struct {
    const int32_t *lengths; /* in  [n] */
    int64_t n;
    int32_t t_block;
    uint64_t seed;
    uint32_t policy; /* 0 = uniform over the unused sequences that fit; 1 = uniform over the LENGTHS (keys of
                        L_dict) that fit and still have an unused sequence; 2 = best fit decreasing, a
                        deterministic comparison strategy that is NOT the paper's rule */
    /* outputs, all caller-allocated */
    int64_t *offsets;         /* [n+1] */
    int32_t *seg_seq;         /* [n]   sequence placed by the k-th draw */
    int32_t *seg_block;       /* [n]   block it went to */
    int32_t *seg_start;       /* [n]   first slot it occupies in that block */
    int32_t *block_seg_begin; /* [n+1] k of the first draw of each block (CSR) */
    int32_t *block_fill;      /* [n]   occupied slots of each block */
    int32_t *seq_block;       /* [n]   inverse: block of sequence i */
    int32_t *seq_start;       /* [n]   inverse: first slot of sequence i */
    /* scalars */
    int64_t n_blocks, sum_t, t_max, first_bad;
    uint64_t checksum;
    int64_t max_segs_per_block;
} oracle_plan_t;

typedef struct { int32_t len; uint32_t h; int32_t id; } ldict_entry_t;

static int ldict_cmp(const void *pa, const void *pb)
{
    const ldict_entry_t *a = (const ldict_entry_t *)pa, *b = (const ldict_entry_t *)pb;
    if (a->len != b->len) return a->len < b->len ? -1 : 1;
    if (a->h != b->h) return a->h < b->h ? -1 : 1;
    if (a->id != b->id) return a->id < b->id ? -1 : 1;
    return 0;
}

static uint64_t fmix64(uint64_t x)
{ /* the 64-bit finaliser of MurmurHash3 (public domain, A. Appleby) */
    x ^= x >> 33; x *= 0xff51afd7ed558ccdULL;
    x ^= x >> 33; x *= 0xc4ceb9fe1a85ec53ULL;
    x ^= x >> 33;
    return x;
}

/* Order-independent 64-bit digest of a segment list (block, start slot, sequence per segment). */
uint64_t oracle_digest(const int32_t *seg_block, const int32_t *seg_start, const int32_t *seg_seq, int64_t n)
{
    uint64_t sum = 0;
    for (int64_t q = 0; q < n; ++q) {
        uint64_t where = ((uint64_t)(uint32_t)seg_block[q] << 32) | (uint64_t)(uint32_t)seg_start[q];
        sum += fmix64(where * 0x9E3779B97F4A7C15ULL + (uint64_t)(uint32_t)seg_seq[q]);
    }
    return sum;
}

int oracle_plan(oracle_plan_t *p)
{
    const int64_t n = p->n;
    const int32_t tb = p->t_block;
    p->n_blocks = 0; p->sum_t = 0; p->t_max = 0; p->first_bad = -1;
    p->checksum = 0; p->max_segs_per_block = 0;
    if (n < 1 || n > 0x7fffffffLL || tb < 1) return ORACLE_ERR_ARG;
    if (p->policy > 2) return ORACLE_ERR_POLICY;

    /* Precondition of the method: 1 <= T_i <= block length. */
    for (int64_t i = 0; i < n; ++i) {
        if (p->lengths[i] < 1 || p->lengths[i] > tb) { p->first_bad = i; return ORACLE_ERR_LENGTH; }
    }
    oracle_offsets(p->lengths, n, p->offsets);
    p->sum_t = p->offsets[n];
    for (int64_t i = 0; i < n; ++i) if (p->lengths[i] > p->t_max) p->t_max = p->lengths[i];

    /* L_dict: for every length, the sequences of that length in (h_i, i) order. */
    ldict_entry_t *dict = (ldict_entry_t *)malloc((size_t)n * sizeof *dict);
    int64_t *first = (int64_t *)calloc((size_t)tb + 2, sizeof *first);  /* first[l]: where length l begins in dict */
    int64_t *unused = (int64_t *)calloc((size_t)tb + 2, sizeof *unused); /* unused[l]: entries of length l not yet drawn */
    if (!dict || !first || !unused) { free(dict); free(first); free(unused); return ORACLE_ERR_NOMEM; }
    for (int64_t i = 0; i < n; ++i) {
        dict[i].len = p->lengths[i];
        dict[i].h = oracle_seq_key(p->seed, i);
        dict[i].id = (int32_t)i;
        unused[p->lengths[i]] += 1;
    }
    qsort(dict, (size_t)n, sizeof *dict, ldict_cmp);
    first[1] = 0;
    for (int32_t l = 1; l <= tb; ++l) first[l + 1] = first[l] + unused[l];

    int64_t k = 0;      /* draws made so far */
    int64_t b = 0;      /* current block */
    if (p->policy == 2) {
        /* Best fit decreasing (textbook bin packing heuristic): sequences in decreasing order of length
         * (the reverse of the L_dict order); each goes to the open block whose free room is the smallest
         * that still holds it -- among blocks with equal room, the one that has had that room longest --
         * or opens a new block when none has room.  head/tail/next: one FIFO of blocks per room value. */
        int32_t *head = (int32_t *)malloc(sizeof(int32_t) * ((size_t)tb + 1));
        int32_t *tail = (int32_t *)malloc(sizeof(int32_t) * ((size_t)tb + 1));
        int32_t *next = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        int32_t *item_block = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        int32_t *item_start = (int32_t *)malloc(sizeof(int32_t) * (size_t)n);
        if (!head || !tail || !next || !item_block || !item_start) {
            free(head); free(tail); free(next); free(item_block); free(item_start);
            free(dict); free(first); free(unused);
            return ORACLE_ERR_NOMEM;
        }
        for (int32_t r = 0; r <= tb; ++r) head[r] = tail[r] = -1;
        for (int64_t t = 0; t < n; ++t) {
            const int32_t l = dict[n - 1 - t].len;
            int32_t r = l;
            while (r <= tb && head[r] < 0) ++r;          /* smallest room >= l among the open blocks */
            int32_t blk, start;
            if (r > tb) { blk = (int32_t)b++; start = 0; r = tb; p->block_fill[blk] = 0; }
            else { blk = head[r]; head[r] = next[blk]; if (head[r] < 0) tail[r] = -1; start = tb - r; }
            const int32_t room = r - l;                   /* a block without room left is never looked at again */
            if (room > 0) {
                next[blk] = -1;
                if (tail[room] >= 0) next[tail[room]] = blk; else head[room] = blk;
                tail[room] = blk;
            }
            item_block[t] = blk; item_start[t] = start;
            p->block_fill[blk] = start + l;
        }
        /* segment list: blocks in opening order, inside a block in placement order */
        for (int64_t q = 0; q <= b; ++q) p->block_seg_begin[q] = 0;
        for (int64_t t = 0; t < n; ++t) p->block_seg_begin[item_block[t] + 1] += 1;
        for (int64_t q = 0; q < b; ++q) {
            if (p->block_seg_begin[q + 1] > p->max_segs_per_block) p->max_segs_per_block = p->block_seg_begin[q + 1];
            p->block_seg_begin[q + 1] += p->block_seg_begin[q];
        }
        int32_t *cursor = next;                           /* reuse: next free position of each block */
        for (int64_t q = 0; q < b; ++q) cursor[q] = p->block_seg_begin[q];
        for (int64_t t = 0; t < n; ++t) {
            const int32_t id = dict[n - 1 - t].id, blk = item_block[t], pos = cursor[blk]++;
            p->seg_seq[pos] = id; p->seg_block[pos] = blk; p->seg_start[pos] = item_start[t];
            p->seq_block[id] = blk; p->seq_start[id] = item_start[t];
        }
        free(head); free(tail); free(next); free(item_block); free(item_start);
        k = n;
    }
    while (k < n) {
        int32_t remaining = tb, start = 0;
        p->block_seg_begin[b] = (int32_t)k;
        for (;;) {
            int32_t l = 1;
            if (p->policy == 0) {
                /* m: unused sequences that still fit */
                int64_t m = 0;
                for (int32_t q = 1; q <= remaining; ++q) m += unused[q];
                if (m == 0) break;
                /* Random_*(): the j-th of them, counted in order of length */
                uint64_t j = oracle_pick(oracle_draw_word(p->seed, k), (uint64_t)m);
                int64_t run = unused[1];
                while ((uint64_t)run <= j) { l += 1; run += unused[l]; }
            } else {
                /* m: keys of L_dict (lengths) that fit and are not exhausted */
                int64_t m = 0;
                for (int32_t q = 1; q <= remaining; ++q) m += unused[q] > 0;
                if (m == 0) break;
                /* Random_*(): the j-th such key in increasing order, then an entry of its list */
                uint64_t j = oracle_pick(oracle_draw_word(p->seed, k), (uint64_t)m);
                int64_t run = unused[1] > 0;
                while ((uint64_t)run <= j) { l += 1; run += unused[l] > 0; }
            }
            /* first unused entry of L_dict[l] */
            int64_t taken = (first[l + 1] - first[l]) - unused[l];
            int32_t id = dict[first[l] + taken].id;
            unused[l] -= 1;
            p->seg_seq[k] = id;
            p->seg_block[k] = (int32_t)b;
            p->seg_start[k] = start;
            p->seq_block[id] = (int32_t)b;
            p->seq_start[id] = start;
            start += l;
            remaining -= l;
            k += 1;
        }
        p->block_fill[b] = start; /* slots [start, t_block) are padding */
        int64_t segs = k - p->block_seg_begin[b];
        if (segs > p->max_segs_per_block) p->max_segs_per_block = segs;
        b += 1;
    }
    if (p->policy != 2) p->block_seg_begin[b] = (int32_t)k;
    p->n_blocks = b;

    p->checksum = oracle_digest(p->seg_block, p->seg_start, p->seg_seq, n);

    free(dict); free(first); free(unused);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Per-slot metadata for blocks [block_begin, block_begin + block_count).     */
/* Blocks at or beyond n_blocks are filler: all padding.                      */
/* ------------------------------------------------------------------------ */
typedef struct {
    int64_t n, n_blocks;
    int32_t t_block;
    const int64_t *offsets;
    const int32_t *seg_seq, *seg_start, *block_seg_begin;
} oracle_tables_t;

int oracle_metadata(const oracle_tables_t *t, int64_t block_begin, int64_t block_count,
                    int32_t *seq_id, int32_t *pos, uint8_t *reset, uint8_t *valid)
{
    if (block_begin < 0 || block_count < 0) return ORACLE_ERR_ARG;
    for (int64_t q = 0; q < block_count; ++q) {
        int64_t b = block_begin + q;
        int32_t *sid = seq_id + q * t->t_block, *ps = pos + q * t->t_block;
        uint8_t *rs = reset + q * t->t_block, *vd = valid + q * t->t_block;
        for (int32_t s = 0; s < t->t_block; ++s) { sid[s] = -1; ps[s] = -1; rs[s] = 0; vd[s] = 0; }
        if (b >= t->n_blocks) continue;
        for (int32_t k = t->block_seg_begin[b]; k < t->block_seg_begin[b + 1]; ++k) {
            int32_t id = t->seg_seq[k];
            int64_t len = t->offsets[id + 1] - t->offsets[id];
            for (int64_t f = 0; f < len; ++f) {
                int64_t s = t->seg_start[k] + f;
                sid[s] = id; ps[s] = (int32_t)f; vd[s] = 1; rs[s] = (f == 0);
            }
        }
    }
    return ORACLE_OK;
}

/* dense[q, s, :] = store[offsets[id] + f, :] on valid slots, pad_byte elsewhere. */
int oracle_pack(const oracle_tables_t *t, const uint8_t *store, int64_t frame_bytes,
                int64_t block_begin, int64_t block_count, uint8_t *dense, uint8_t pad_byte)
{
    if (block_begin < 0 || block_count < 0 || frame_bytes < 1) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            uint8_t *dst = dense + ((size_t)q * (size_t)t->t_block + (size_t)s) * (size_t)frame_bytes;
            if (vd[s]) memcpy(dst, store + (size_t)(t->offsets[sid[s]] + ps[s]) * (size_t)frame_bytes, (size_t)frame_bytes);
            else memset(dst, pad_byte, (size_t)frame_bytes);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* The other padding the paper mentions (caption of its naive-padding figure: "adding 0's or repeating the
 * last entry of the sequence"), applied to blocks: the padding slots of a block repeat the frame in the
 * block's last occupied slot.  A filler block holds no frame and is filled with pad_byte. */
int oracle_pack_repeat_last(const oracle_tables_t *t, const uint8_t *store, int64_t frame_bytes,
                            int64_t block_begin, int64_t block_count, uint8_t *dense, uint8_t pad_byte)
{
    int rc = oracle_pack(t, store, frame_bytes, block_begin, block_count, dense, pad_byte);
    if (rc != ORACLE_OK) return rc;
    uint8_t *vd = (uint8_t *)malloc((size_t)t->t_block), *rs = (uint8_t *)malloc((size_t)t->t_block);
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        int32_t last = -1;
        for (int32_t s = 0; s < t->t_block; ++s) if (vd[s]) last = s;
        if (last < 0) continue;
        uint8_t *row = dense + (size_t)q * (size_t)t->t_block * (size_t)frame_bytes;
        for (int32_t s = last + 1; s < t->t_block; ++s)
            memcpy(row + (size_t)s * (size_t)frame_bytes, row + (size_t)last * (size_t)frame_bytes, (size_t)frame_bytes);
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* ragged_out[offsets[id] + f, :] = dense_out[q, s, :] on valid slots; padding ignored. */
int oracle_unpack(const oracle_tables_t *t, const uint8_t *dense_out, int64_t frame_bytes,
                  int64_t block_begin, int64_t block_count, uint8_t *ragged_out)
{
    if (block_begin < 0 || block_count < 0 || frame_bytes < 1) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            if (!vd[s]) continue;
            memcpy(ragged_out + (size_t)(t->offsets[sid[s]] + ps[s]) * (size_t)frame_bytes,
                   dense_out + ((size_t)q * (size_t)t->t_block + (size_t)s) * (size_t)frame_bytes, (size_t)frame_bytes);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Frames whose size differs from sample to sample (problem statement: every   */
/* sample has its own H, W and T).  Sequence i holds T_i frames of F_i bytes,  */
/* back to back, at byte_offsets[i] of the store; a slot of a block has room   */
/* for the largest frame and a smaller frame is followed by padding.           */
/* ------------------------------------------------------------------------ */
void oracle_byte_offsets(const int32_t *lengths, const int32_t *frame_bytes, int64_t n, int64_t *byte_offsets)
{
    int64_t run = 0;
    for (int64_t i = 0; i < n; ++i) { byte_offsets[i] = run; run += (int64_t)lengths[i] * (int64_t)frame_bytes[i]; }
    byte_offsets[n] = run;
}

int oracle_pack_var(const oracle_tables_t *t, const uint8_t *store, const int32_t *frame_bytes,
                    const int64_t *byte_offsets, int64_t slot_bytes, int64_t block_begin, int64_t block_count,
                    uint8_t *dense, uint8_t pad_byte)
{
    if (block_begin < 0 || block_count < 0 || slot_bytes < 1) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < t->n; ++i) if (frame_bytes[i] < 1 || frame_bytes[i] > slot_bytes) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            uint8_t *dst = dense + ((size_t)q * (size_t)t->t_block + (size_t)s) * (size_t)slot_bytes;
            size_t have = 0;
            if (vd[s]) {
                have = (size_t)frame_bytes[sid[s]];
                memcpy(dst, store + (size_t)byte_offsets[sid[s]] + (size_t)ps[s] * have, have);
            }
            memset(dst + have, pad_byte, (size_t)slot_bytes - have);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

int oracle_unpack_var(const oracle_tables_t *t, const uint8_t *dense_out, const int32_t *frame_bytes,
                      const int64_t *byte_offsets, int64_t slot_bytes, int64_t block_begin, int64_t block_count,
                      uint8_t *ragged_out)
{
    if (block_begin < 0 || block_count < 0 || slot_bytes < 1) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < t->n; ++i) if (frame_bytes[i] < 1 || frame_bytes[i] > slot_bytes) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            if (!vd[s]) continue;
            size_t have = (size_t)frame_bytes[sid[s]];
            memcpy(ragged_out + (size_t)byte_offsets[sid[s]] + (size_t)ps[s] * have,
                   dense_out + ((size_t)q * (size_t)t->t_block + (size_t)s) * (size_t)slot_bytes, have);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* Frames as images of rows_i rows of row_bytes_i bytes (H_i x W_i of the problem statement): a slot is a
 * canvas of rows_max rows of row_stride bytes, an image sits in its top left corner, the rest is padding.
 * Sequence i holds T_i images of rows_i * row_bytes_i bytes back to back at byte_offsets[i]. */
void oracle_byte_offsets2d(const int32_t *lengths, const int32_t *rows, const int32_t *row_bytes, int64_t n,
                           int64_t *byte_offsets)
{
    int64_t run = 0;
    for (int64_t i = 0; i < n; ++i) {
        byte_offsets[i] = run;
        run += (int64_t)lengths[i] * (int64_t)rows[i] * (int64_t)row_bytes[i];
    }
    byte_offsets[n] = run;
}

static int var2d_args_ok(const oracle_tables_t *t, const int32_t *rows, const int32_t *row_bytes, int64_t rows_max,
                         int64_t row_stride)
{
    if (rows_max < 1 || row_stride < 1) return 0;
    for (int64_t i = 0; i < t->n; ++i)
        if (rows[i] < 1 || rows[i] > rows_max || row_bytes[i] < 1 || row_bytes[i] > row_stride) return 0;
    return 1;
}

int oracle_pack_var2d(const oracle_tables_t *t, const uint8_t *store, const int32_t *rows, const int32_t *row_bytes,
                      const int64_t *byte_offsets, int64_t rows_max, int64_t row_stride, int64_t block_begin,
                      int64_t block_count, uint8_t *dense, uint8_t pad_byte)
{
    if (block_begin < 0 || block_count < 0 || !var2d_args_ok(t, rows, row_bytes, rows_max, row_stride)) return ORACLE_ERR_ARG;
    const size_t canvas = (size_t)rows_max * (size_t)row_stride;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            uint8_t *dst = dense + ((size_t)q * (size_t)t->t_block + (size_t)s) * canvas;
            memset(dst, pad_byte, canvas);
            if (!vd[s]) continue;
            const size_t h = (size_t)rows[sid[s]], w = (size_t)row_bytes[sid[s]];
            const uint8_t *img = store + (size_t)byte_offsets[sid[s]] + (size_t)ps[s] * h * w;
            for (size_t r = 0; r < h; ++r) memcpy(dst + r * (size_t)row_stride, img + r * w, w);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

int oracle_unpack_var2d(const oracle_tables_t *t, const uint8_t *dense_out, const int32_t *rows, const int32_t *row_bytes,
                        const int64_t *byte_offsets, int64_t rows_max, int64_t row_stride, int64_t block_begin,
                        int64_t block_count, uint8_t *ragged_out)
{
    if (block_begin < 0 || block_count < 0 || !var2d_args_ok(t, rows, row_bytes, rows_max, row_stride)) return ORACLE_ERR_ARG;
    const size_t canvas = (size_t)rows_max * (size_t)row_stride;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            if (!vd[s]) continue;
            const uint8_t *src = dense_out + ((size_t)q * (size_t)t->t_block + (size_t)s) * canvas;
            const size_t h = (size_t)rows[sid[s]], w = (size_t)row_bytes[sid[s]];
            uint8_t *img = ragged_out + (size_t)byte_offsets[sid[s]] + (size_t)ps[s] * h * w;
            for (size_t r = 0; r < h; ++r) memcpy(img + r * w, src + r * (size_t)row_stride, w);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Consumer side of the start table (Methods, second paragraph): a recurrent  */
/* model feeds information of frame t-1 into frame t and must discard it       */
/* wherever a new sequence starts inside a block.                              */
/* ------------------------------------------------------------------------ */

/* prev[q, s, :] = dense[q, s-1, :] where slot s holds frame f >= 1 of a sequence (the frame before
 * it belongs to the same sequence); fill_byte where it holds a first frame, padding, or the block
 * is filler.  This is "what frame t receives from frame t-1" for a whole batch at once. */
int oracle_carry_prev(const oracle_tables_t *t, const uint8_t *dense, int64_t frame_bytes,
                      int64_t block_begin, int64_t block_count, uint8_t *prev, uint8_t fill_byte)
{
    if (block_begin < 0 || block_count < 0 || frame_bytes < 1) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s) {
            size_t at = ((size_t)q * (size_t)t->t_block + (size_t)s) * (size_t)frame_bytes;
            if (vd[s] && !rs[s]) memcpy(prev + at, dense + at - (size_t)frame_bytes, (size_t)frame_bytes);
            else memset(prev + at, fill_byte, (size_t)frame_bytes);
        }
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* One step of a recurrence that walks the slots of a batch in order: before slot `slot` is
 * processed, row q of the carried state is replaced by `init` (zeros when init is NULL) unless a
 * sequence continues at that slot, i.e. on a first frame, on padding and in filler blocks.
 * Rows whose sequence continues are left as they are. */
int oracle_reset_state(const oracle_tables_t *t, int64_t block_begin, int64_t block_count, int32_t slot,
                       uint8_t *state, int64_t state_bytes, const uint8_t *init)
{
    if (block_begin < 0 || block_count < 0 || state_bytes < 1 || slot < 0 || slot >= t->t_block) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        if (vd[slot] && !rs[slot]) continue;
        if (init) memcpy(state + (size_t)q * (size_t)state_bytes, init, (size_t)state_bytes);
        else memset(state + (size_t)q * (size_t)state_bytes, 0, (size_t)state_bytes);
    }
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* Sum (in double precision, slot order) and count of per-slot float values over the frames of the
 * given blocks; padding and filler blocks contribute nothing (a loss must not see them). */
int oracle_valid_sum(const oracle_tables_t *t, int64_t block_begin, int64_t block_count, const float *values,
                     double *sum, int64_t *count)
{
    if (block_begin < 0 || block_count < 0) return ORACLE_ERR_ARG;
    int32_t *sid = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    int32_t *ps = (int32_t *)malloc(sizeof(int32_t) * (size_t)t->t_block);
    uint8_t *rs = (uint8_t *)malloc((size_t)t->t_block), *vd = (uint8_t *)malloc((size_t)t->t_block);
    if (!sid || !ps || !rs || !vd) { free(sid); free(ps); free(rs); free(vd); return ORACLE_ERR_NOMEM; }
    double acc = 0.0;
    int64_t cnt = 0;
    for (int64_t q = 0; q < block_count; ++q) {
        oracle_metadata(t, block_begin + q, 1, sid, ps, rs, vd);
        for (int32_t s = 0; s < t->t_block; ++s)
            if (vd[s]) { acc += (double)values[(size_t)q * (size_t)t->t_block + (size_t)s]; ++cnt; }
    }
    *sum = acc; *count = cnt;
    free(sid); free(ps); free(rs); free(vd);
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* Padding statistics (closed forms).                                         */
/*   naive  : every sample padded to the longest one: N*T_max - sum T         */
/*   packed : n_blocks*T_block - sum T                                         */
/* ------------------------------------------------------------------------ */
typedef struct {
    int64_t n, sum_t, t_max, t_block, n_blocks;
    int64_t pad_packed, pad_naive_tmax, pad_naive_tblock, min_blocks;
    double frac_packed, frac_naive_tmax, frac_naive_tblock, reduction_vs_tmax, mean_segs_per_block;
} oracle_stats_t;

int oracle_stats(oracle_stats_t *s)
{
    if (s->n < 1 || s->t_block < 1 || s->sum_t < 1 || s->n_blocks < 0) return ORACLE_ERR_ARG;
    s->pad_packed = s->n_blocks * s->t_block - s->sum_t;
    s->pad_naive_tmax = s->n * s->t_max - s->sum_t;
    s->pad_naive_tblock = s->n * s->t_block - s->sum_t;
    s->min_blocks = (s->sum_t + s->t_block - 1) / s->t_block;
    s->frac_packed = s->n_blocks ? (double)s->pad_packed / (double)(s->n_blocks * s->t_block) : 0.0;
    s->frac_naive_tmax = s->t_max ? (double)s->pad_naive_tmax / (double)(s->n * s->t_max) : 0.0;
    s->frac_naive_tblock = (double)s->pad_naive_tblock / (double)(s->n * s->t_block);
    s->reduction_vs_tmax = s->pad_packed > 0 ? (double)s->pad_naive_tmax / (double)s->pad_packed : 0.0;
    s->mean_segs_per_block = s->n_blocks ? (double)s->n / (double)s->n_blocks : 0.0;
    return ORACLE_OK;
}

/* ------------------------------------------------------------------------ */
/* The chunking strategy the paper compares with (section "Problem Statement  */
/* and Current Limitations": each sample is broken into chunks of T_block      */
/* frames and each chunk is treated as an individual sample; figure "Sampling  */
/* solution"; Table I, column "sampling": no padding, frames deleted).         */
/* Sequence i is cut at frames 0, c, 2c, ...  With tail == 0 the last, shorter */
/* chunk is kept (and padded when it becomes a block); with tail == 1 only     */
/* full chunks are kept and the remaining T_i mod c frames are deleted, which  */
/* is the reading that gives the table's zero padding.  Chunks are listed in   */
/* order of (sequence, position); chunk j becomes block j.                     */
/* ------------------------------------------------------------------------ */
typedef struct {
    const int32_t *lengths;
    int64_t n;
    int32_t t_chunk;
    uint32_t tail;
    int64_t capacity;      /* room in the three arrays below (0 with NULL arrays: count only) */
    int32_t *chunk_seq;    /* sequence the chunk was cut from */
    int32_t *chunk_first;  /* its first frame inside that sequence */
    int32_t *chunk_len;    /* its frames, 1..t_chunk */
    int64_t n_chunks, frames_kept, frames_deleted, pad_frames, sum_t, t_max, first_bad;
} oracle_chunks_t;

int oracle_chunks(oracle_chunks_t *p)
{
    p->n_chunks = p->frames_kept = p->frames_deleted = p->pad_frames = p->sum_t = p->t_max = 0;
    p->first_bad = -1;
    if (p->n < 1 || p->t_chunk < 1 || p->tail > 1) return ORACLE_ERR_ARG;
    for (int64_t i = 0; i < p->n; ++i)
        if (p->lengths[i] < 1) { p->first_bad = i; return ORACLE_ERR_LENGTH; }
    for (int64_t i = 0; i < p->n; ++i) {
        int32_t t = p->lengths[i];
        p->sum_t += t;
        if (t > p->t_max) p->t_max = t;
        for (int32_t first = 0; first < t; first += p->t_chunk) {
            int32_t len = t - first < p->t_chunk ? t - first : p->t_chunk;
            if (len < p->t_chunk && p->tail == 1) { p->frames_deleted += len; continue; }
            if (p->chunk_seq) {
                if (p->n_chunks >= p->capacity) return ORACLE_ERR_ARG;
                p->chunk_seq[p->n_chunks] = (int32_t)i;
                p->chunk_first[p->n_chunks] = first;
                p->chunk_len[p->n_chunks] = len;
            }
            p->n_chunks += 1;
            p->frames_kept += len;
            p->pad_frames += p->t_chunk - len;
        }
    }
    return ORACLE_OK;
}

typedef struct {
    int64_t n_chunks;
    int32_t t_chunk;
    const int64_t *offsets;   /* of the ORIGINAL sequences in the store */
    const int32_t *chunk_seq, *chunk_first, *chunk_len;
} oracle_chunk_tables_t;

/* Every chunk is a sample of its own: its id is the chunk number, positions count from the chunk's first frame. */
int oracle_chunk_metadata(const oracle_chunk_tables_t *t, int64_t block_begin, int64_t block_count,
                          int32_t *seq_id, int32_t *pos, uint8_t *reset, uint8_t *valid)
{
    if (block_begin < 0 || block_count < 0) return ORACLE_ERR_ARG;
    for (int64_t q = 0; q < block_count; ++q) {
        int64_t j = block_begin + q;
        for (int32_t s = 0; s < t->t_chunk; ++s) {
            int64_t o = q * t->t_chunk + s;
            int is_frame = j < t->n_chunks && s < t->chunk_len[j];
            seq_id[o] = is_frame ? (int32_t)j : -1;
            pos[o] = is_frame ? s : -1;
            reset[o] = (uint8_t)(is_frame && s == 0);
            valid[o] = (uint8_t)is_frame;
        }
    }
    return ORACLE_OK;
}

int oracle_chunk_pack(const oracle_chunk_tables_t *t, const uint8_t *store, int64_t frame_bytes, int64_t block_begin,
                      int64_t block_count, uint8_t *dense, uint8_t pad_byte)
{
    if (block_begin < 0 || block_count < 0 || frame_bytes < 1) return ORACLE_ERR_ARG;
    for (int64_t q = 0; q < block_count; ++q) {
        int64_t j = block_begin + q;
        for (int32_t s = 0; s < t->t_chunk; ++s) {
            uint8_t *dst = dense + ((size_t)q * (size_t)t->t_chunk + (size_t)s) * (size_t)frame_bytes;
            if (j < t->n_chunks && s < t->chunk_len[j]) {
                int64_t frame = t->offsets[t->chunk_seq[j]] + t->chunk_first[j] + s;
                memcpy(dst, store + (size_t)frame * (size_t)frame_bytes, (size_t)frame_bytes);
            } else {
                memset(dst, pad_byte, (size_t)frame_bytes);
            }
        }
    }
    return ORACLE_OK;
}

/* Frames that the strategy deleted have no slot anywhere and stay untouched in ragged_out. */
int oracle_chunk_unpack(const oracle_chunk_tables_t *t, const uint8_t *dense_out, int64_t frame_bytes, int64_t block_begin,
                        int64_t block_count, uint8_t *ragged_out)
{
    if (block_begin < 0 || block_count < 0 || frame_bytes < 1) return ORACLE_ERR_ARG;
    for (int64_t q = 0; q < block_count; ++q) {
        int64_t j = block_begin + q;
        if (j >= t->n_chunks) continue;
        for (int32_t s = 0; s < t->chunk_len[j]; ++s) {
            int64_t frame = t->offsets[t->chunk_seq[j]] + t->chunk_first[j] + s;
            memcpy(ragged_out + (size_t)frame * (size_t)frame_bytes,
                   dense_out + ((size_t)q * (size_t)t->t_chunk + (size_t)s) * (size_t)frame_bytes, (size_t)frame_bytes);
        }
    }
    return ORACLE_OK;
}

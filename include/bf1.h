/*
 * bf1.h -- C ABI of the BF1 causal dyadic block-sparse attention forward (prefill) library
 *          for NVIDIA B200 (sm_100a).
 *
 * The operator (paper Section 3.1): a sequence of n tokens is cut into B = ceil(n / b)
 * blocks of width b.  Query block j attends, with exact softmax, to the keys of the blocks
 *
 *        P(j) = {j, j-1, j-2, 0} u {j - 2^r : r >= 2}        (Eq. 1)
 *
 * with invalid and duplicate indices removed; inside the self block the token-level causal
 * triangle applies, every other selected block is strictly earlier and is read in full.
 * No score bias is used.  Proposition 1 bounds |P(j)| by 4 + floor(log2 j), which makes the
 * selected token pairs O(n log n).
 *
 * Conventions for every entry point
 *   - C linkage, plain pointers and sizes, int status return (bf1_status); no exceptions.
 *   - "dev" pointers are CUDA device pointers owned by the caller; "host" pointers are
 *     ordinary host memory.  The library allocates no device memory.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*; NULL = default
 *     stream) and return without synchronising.  Host-checkable argument errors are
 *     reported before anything is launched.  Errors that only the device can see are
 *     OR-ed into the route's `status` word (see BF1_DEV_* below), never a trap.
 *   - Tensors are packed over the batch ("varlen"): Q and O are [T, Hq, d], K and V are
 *     [T, Hkv, d], bf16, row-major, T = total tokens; sequence s owns token rows
 *     cu_seqlens[s] .. cu_seqlens[s+1]-1.  With equal lengths this is [B, n, H, d].
 *     LSE is fp32 [Hq, T].  Every sequence is cut into blocks from its own first token and
 *     never attends across a sequence boundary.
 *   - GQA: Hq = G * Hkv; query head h reads KV head floor(h / G) (the paper gives only the
 *     head counts, Section 4.1; this is the usual grouped convention).
 *   - Base pointers of Q, K, V, O must be 16-byte aligned.
 *   - Supported geometry, in every entry point: b = 64 (Section 3.1), d in {64, 128},
 *     G = hq / hkv in {1, 2, 4} (Section 4.1's model has 16 query / 8 KV heads, G = 2).
 *     Anything else returns BF1_ERR_UNSUPPORTED.
 */
#ifndef BF1_H_
#define BF1_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    BF1_OK = 0,
    BF1_ERR_INVALID_ARG = -1,   /* null pointer, negative size, misaligned pointer, ...   */
    BF1_ERR_UNSUPPORTED = -2,   /* geometry outside the supported set                     */
    BF1_ERR_CAPACITY = -3,      /* route buffers too small for this batch                 */
    BF1_ERR_CUDA = -4,          /* a CUDA runtime / driver call failed                    */
    BF1_ERR_NO_DEVICE = -5      /* no usable sm_100 device                                */
} bf1_status;

/* Bits OR-ed into *route.status by device code. */
enum {
    BF1_DEV_BAD_SEQLENS = 1,    /* cu_seqlens not non-decreasing from 0 to total_tokens,
                                   or a sequence longer than max_seqlen                   */
    BF1_DEV_CAPACITY = 2,       /* more query blocks, or a longer list, than the buffers  */
    BF1_DEV_WAIT_TIMEOUT = 4,   /* a bounded on-chip wait gave up (should never happen)   */
    BF1_DEV_BAD_ROUTE = 8       /* attention kernel met a list entry outside [0, j]       */
};

/* Route parameters.  The paper's reported configuration (Section 3.1) is
 * {64, 2, 1, 1}: two local predecessor blocks, the global first block, dyadic
 * predecessors.  `dyadic` adds j - 2^k for every k >= 0 with j - 2^k >= 0; with
 * local_blocks = 2 this is Eq. 1's "r >= 2" set, because 2^0 and 2^1 are the local blocks. */
typedef struct {
    int32_t block;         /* b: 64 (the paper's) or 128, see below                      */
    int32_t local_blocks;  /* W >= 0                                                     */
    int32_t global_first;  /* 0 or 1                                                     */
    int32_t dyadic;        /* 0 or 1                                                     */
} bf1_route_cfg;

/* Block width.  Every array of a route is kept per TILE of 64 tokens, whatever b is, and the
 * kernels only ever see tiles.  With b = 64 a tile is a block.  With b = 128, tile t of a sequence
 * belongs to block j = t / 2; its list holds both tiles of every earlier block of P(j) and the
 * tiles of block j up to t itself, which selects, token for token, what Eq. 1 selects at b = 128
 * (earlier blocks in full, the causal triangle inside the self block).  "Query block", "block
 * index" and "list" below therefore mean tiles and tile indices; bf1_route_capacity returns the
 * tile count and twice the block-level list length.  The sequence-sharded prefill takes b = 64 only.
 *
 * A planned route: for every query block of every sequence, the ascending list of KV
 * block indices it reads (sequence-local; the last entry is the query block itself), the
 * list length, and the number of selected token pairs (Proposition 1's accounting: a
 * non-self block gives rows*b pairs, the self block rows*(rows+1)/2, rows = tokens in the
 * query block).  Query blocks are numbered sequence by sequence ("slots").
 * The two capacities are host values; every pointer is device memory owned by the caller. */
typedef struct {
    int32_t  capacity_qblocks; /* slots available in the arrays below                     */
    int32_t  max_degree;       /* row pitch of kv_idx                                     */
    int32_t *qb_seq;           /* [capacity] sequence of the slot                         */
    int32_t *qb_block;         /* [capacity] block index j inside that sequence           */
    int32_t *kv_count;         /* [capacity] |P(j)|                                       */
    int32_t *kv_idx;           /* [capacity, max_degree] ascending; unused entries = -1   */
    int32_t *pair_count;       /* [capacity] selected token pairs of the slot             */
    int32_t *order;            /* [capacity] slots sorted by descending kv_count: the
                                  order in which the attention kernel hands out work      */
    int64_t *total_pairs;      /* [1] sum of pair_count                                   */
    int32_t *num_qblocks;      /* [1] slots actually used                                 */
    int32_t *status;           /* [1] BF1_DEV_* bits; 0 = fine.  Written (not OR-ed) by
                                  bf1_plan_route, OR-ed by the attention entry points     */
    int32_t *sched;            /* [2] work hand-out counters of the attention kernel: zeroed
                                  by bf1_plan_route and put back to zero by every
                                  bf1_attn_fwd launch when it finishes.  Launches that share
                                  a route must therefore be ordered (same stream, or
                                  otherwise not overlapping on the GPU)                    */
} bf1_route;

/* Host-only helper: how large the route arrays must be for a batch of `batch` sequences,
 * `total_tokens` tokens in all, none longer than `max_seqlen`.  capacity_qblocks is the
 * largest value sum_s ceil(n_s / b) can take for that batch size and token total (exact for
 * batch = 1); max_degree is the largest |P(j)| any block of a
 * sequence of max_seqlen tokens has (Proposition 1).  Touches no device. */
int bf1_route_capacity(int32_t batch, int64_t total_tokens, int32_t max_seqlen,
                       const bf1_route_cfg *cfg /* host */,
                       int32_t *capacity_qblocks /* host out */, int32_t *max_degree /* host out */);

/* Eq. 1 on the device: fills every array of `out` from cu_seqlens.  One small kernel; meant
 * to run once per (sequence lengths, cfg) and be reused by every layer.
 *   cu_seqlens_dev  [batch+1] int32 device, cu_seqlens[0] = 0, cu_seqlens[batch] = total_tokens
 *   out             host struct holding device pointers (see bf1_route)
 * Device-side validation failures set *out->status and leave num_qblocks = 0. */
int bf1_plan_route(const int32_t *cu_seqlens_dev, int32_t batch, int64_t total_tokens,
                   int32_t max_seqlen, const bf1_route_cfg *cfg /* host */,
                   const bf1_route *out /* host struct, device arrays */, void *stream);

/* BF1 forward (Section 3.1): for every query block, online-softmax attention over exactly
 * the KV blocks its list names, causal triangle on the self block.
 *   q, k, v   device bf16, [T, hq, d], [T, hkv, d], [T, hkv, d]
 *   softmax_scale  scores are scale * <q, k>; <= 0 selects 1 / sqrt(d)
 *   route     a route planned for the same cu_seqlens (any lists of distinct earlier blocks
 *             whose last entry is the query block itself are accepted, so other block-sparse
 *             causal routes can be run through the same kernel; the planners write the
 *             earlier blocks in ascending order, the kernel does not depend on it)
 *   o         device bf16 [T, hq, d], written for every token row
 *   lse       device fp32 [hq, T]: natural log of the sum of exp(scaled scores) over the
 *             selected keys
 * Rows of o/lse outside every sequence are not touched. */
int bf1_attn_fwd(const void *q, const void *k, const void *v, const int32_t *cu_seqlens_dev,
                 int32_t batch, int64_t total_tokens, int32_t max_seqlen, int32_t hq,
                 int32_t hkv, int32_t d, float softmax_scale, const bf1_route *route /* host */,
                 void *o, float *lse, void *stream);

/* Dense causal attention through the same kernel (every predecessor block selected):
 * the paper's dense comparator (Section 4.3) and its dense-path equivalence gate
 * (Section 4.2).  Arguments as bf1_attn_fwd without the route.  `work_dev` is an optional
 * [4] int32 device array, all zero before its first use: word 0 receives BF1_DEV_* bits,
 * words 1..2 are the work hand-out counters (left at zero by every launch; launches sharing
 * the array must be ordered), word 3 is reserved.  NULL selects a static work split and
 * drops device-side error reporting. */
int bf1_dense_causal_fwd(const void *q, const void *k, const void *v,
                         const int32_t *cu_seqlens_dev, int32_t batch, int64_t total_tokens,
                         int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d,
                         float softmax_scale, void *o, float *lse, int32_t *work_dev,
                         void *stream);

/* (The paper has no counterpart for this entry point; it exists for callers of this library.)
 * BF1 forward for callers that cannot allocate device memory: code running after a server has
 * fixed its memory budget, inside a real-time loop, or under an allocator that must not be
 * re-entered.  It does what bf1_plan_route followed by bf1_attn_fwd do, but keeps the route
 * arrays and the kernel's work hand-out counters in a fixed array inside the library (about
 * 0.6 MB of device memory on every GPU that loads the library, held until the process exits),
 * so the caller passes only inputs and outputs.
 *   cfg         host; route parameters as for bf1_plan_route
 *   status_dev  optional [1] int32 device word that receives the BF1_DEV_* bits (written by the
 *               planner, OR-ed by the attention kernel); NULL keeps them inside the library
 *   other arguments as bf1_attn_fwd
 * Limits: the batch may hold at most 4096 query blocks and lists of at most 32 entries (the
 * paper's route needs 3 + floor(log2(B-1))).  The block count is checked on the host through
 * bf1_route_capacity's upper bound for (batch, total_tokens): one sequence of 262,144 tokens
 * (exactly 4096 blocks) is accepted, a batch of B sequences may hold 64 * (4096 - B) + B tokens.
 * Beyond that the call returns BF1_ERR_CAPACITY and launches nothing; so do host-checkable
 * argument errors, before the planner runs.  With status_dev == NULL a device-side refusal
 * (BF1_DEV_BAD_SEQLENS from the planner, which then leaves o and lse unwritten) cannot be read
 * back by the caller: pass a status word when the lengths are not trusted.  It calls no cudaMalloc / cudaFree / allocating library routine.  The first call on a
 * device looks up the array's address; make it before any stream capture.  All calls share the
 * array and overwrite the previous call's contents, so calls that may overlap on the GPU
 * (streams without ordering between them) race and must be avoided. */
int bf1_attn_fwd_noalloc(const void *q, const void *k, const void *v, const int32_t *cu_seqlens_dev,
                         int32_t batch, int64_t total_tokens, int32_t max_seqlen, int32_t hq,
                         int32_t hkv, int32_t d, float softmax_scale,
                         const bf1_route_cfg *cfg /* host */, void *o, float *lse,
                         int32_t *status_dev, void *stream);

/* ---- cached one-token decode over selected KV pages (Section 3.2, Section 5.4) -----------------
 * The newest token of a sequence with n cached tokens (position n-1, block j = (n-1)/64) attends to
 * the pages of P(j), the self page only up to token n-1: O(log B) pages per step.  The KV cache is
 * paged: k_pages / v_pages are [num_pages, 64, hkv, d] bf16 and page_table[s, i] names the
 * physical page that holds logical block i of sequence s.  The page list changes only when n
 * crosses a block boundary, so one plan serves a whole 64-token route epoch (Section 5.4 names
 * keeping a plan alive across such an epoch as the open systems problem).  Pages stay 64 tokens
 * with b = 128: a listed block is then two pages, the newest token's own block its pages up to the
 * one that holds the token, and a plan still serves 64 tokens. */
typedef struct {
    int32_t  max_degree;   /* host: row pitch of `page`                                          */
    int32_t *count;        /* [batch] pages to read for the sequence (0 for an empty sequence)   */
    int32_t *page;         /* [batch, max_degree] physical pages in ascending logical-block
                              order, the self page last; unused entries = -1                     */
    int32_t *block;        /* [batch] block index j the plan was made for (-1 if empty)          */
    int32_t *status;       /* [1] BF1_DEV_* bits; written by bf1_plan_decode, OR-ed by the
                              attention call                                                     */
} bf1_decode_plan;         /* all pointers: device memory owned by the caller                    */

/* Eq. 1 for the newest token's block of every sequence, mapped through the page table.
 *   seqlens_dev     [batch] int32 device: cached tokens per sequence (0 allowed)
 *   page_table_dev  [batch, max_pages_per_seq] int32 device
 * A sequence that needs a logical block >= max_pages_per_seq sets BF1_DEV_BAD_SEQLENS. */
int bf1_plan_decode(const int32_t *seqlens_dev, const int32_t *page_table_dev,
                    int32_t max_pages_per_seq, int32_t batch, const bf1_route_cfg *cfg /* host */,
                    const bf1_decode_plan *out /* host struct, device arrays */, void *stream);

/* Bytes of device scratch bf1_decode_fwd needs (partial results of the split over pages and one
 * ticket word per sequence, KV head and pair of query heads).  Host only; -1 on bad arguments. */
int64_t bf1_decode_workspace_bytes(int32_t batch, int32_t hq, int32_t hkv, int32_t max_degree,
                                   int32_t d);

/* One decode step for every sequence of the batch.
 *   q            device bf16 [batch, hq, d]: the newest token's queries
 *   seqlens_dev  [batch] current cached lengths INCLUDING the newest token; must lie in the block
 *                the plan was made for, otherwise BF1_DEV_BAD_ROUTE is set and the sequence skipped
 *   workspace    device, 16-byte aligned, bf1_decode_workspace_bytes() bytes, all zero before the
 *                first call; every call leaves its ticket words at zero again, so it can be
 *                reused by calls that do not overlap on the GPU
 *   o            device bf16 [batch, hq, d];  lse  device fp32 [hq, batch]
 * Rows of empty sequences are not written.  Geometry limits as for bf1_attn_fwd. */
int bf1_decode_fwd(const void *q, const void *k_pages, const void *v_pages, int32_t num_pages,
                   const int32_t *seqlens_dev, int32_t batch, int32_t hq, int32_t hkv, int32_t d,
                   float softmax_scale, const bf1_decode_plan *plan /* host */, void *workspace,
                   void *o, float *lse, void *stream);

/* ---- backward over the same route (Section 4.2's gates include a backward pass with finite
 * Q, K and V gradients) ---------------------------------------------------------------------------
 * Given the forward's inputs, its outputs o and lse, and the upstream gradient d_o [T, hq, d] bf16,
 * writes dq [T, hq, d], dk and dv [T, hkv, d] in bf16 (the gradients of the G query heads of a KV
 * head add up in dk, dv).  P is recomputed as exp(scale * <q, k> - lse).  dq is computed along the
 * route (one query block at a time over its list), dk and dv along the inverse route (one KV block
 * at a time over the query blocks that read it), which the call derives from the lists itself: no
 * floating-point atomics anywhere, so all three gradients come out bit-identical on every run.
 * `workspace` (bf1_attn_bwd_workspace_bytes() bytes, 256-byte aligned, contents irrelevant on entry)
 * holds the row terms <d_o, o>, the inverse route and the partial sums of KV blocks with very many
 * readers.  Geometry limits as bf1_attn_fwd.  `route` must be the forward's (host struct; only its
 * capacities are used by the size helper). */
int64_t bf1_attn_bwd_workspace_bytes(const bf1_route *route /* host */, int64_t total_tokens,
                                     int32_t hq, int32_t hkv, int32_t d);
int bf1_attn_bwd(const void *q, const void *k, const void *v, const void *o, const float *lse,
                 const void *d_o, const int32_t *cu_seqlens_dev, int32_t batch, int64_t total_tokens,
                 int32_t max_seqlen, int32_t hq, int32_t hkv, int32_t d, float softmax_scale,
                 const bf1_route *route /* host */, void *workspace, void *dq, void *dk, void *dv,
                 void *stream);

/* ---- sequence-sharded prefill ----------------------------------------------------------------------
 * One long sequence cut into contiguous shards of whole blocks, one shard per GPU.  The route is
 * "block aligned and data independent" (Section 3.1), so the KV blocks a shard reads from earlier shards
 * -- block 0, the two blocks in front of it, and the dyadic predecessors j - 2^k of its query blocks
 * that fall in front of it: O(shard blocks x log B) blocks, Proposition 1 -- are known at plan time,
 * before any tensor exists.  The exchange itself is left to the caller's communication library (plain
 * point-to-point copies into a landing buffer in the receiver's own memory); the library provides the
 * two plans:
 *
 * bf1_shard_needed_blocks (host only): the ascending global indices of the KV blocks that the shard
 * of query blocks [lo_block, hi_block) reads but does not own (all are < lo_block).  Returns
 * BF1_ERR_CAPACITY when `capacity` entries are not enough (count_out still receives the number).
 *
 * bf1_plan_route_shard (device): the shard's route over its LOCAL key/value tensor, which the caller
 * lays out as [the needed blocks in ascending global order | the shard's own blocks], 64 token rows
 * per block ("virtual sequence").  Query, output and LSE tensors use the same row numbering (their
 * first num_needed * 64 rows are never touched).  Lists are re-indexed into that layout: entries stay
 * ascending and end in the query block itself, so bf1_attn_fwd runs the shard unchanged, with
 * cu_seqlens_out_dev = {0, num_needed * 64 + the shard's tokens} written by this call.  Counts and
 * totals are the shard's share of the sequence's selected pairs.  A block of some list that is
 * neither owned nor in `needed_blocks_dev` sets BF1_DEV_BAD_ROUTE in *out->status. */
int bf1_shard_needed_blocks(int64_t n_tokens, const bf1_route_cfg *cfg /* host */, int32_t lo_block,
                            int32_t hi_block, int32_t *blocks_out /* host */, int32_t capacity,
                            int32_t *count_out /* host */);
int bf1_plan_route_shard(int64_t n_tokens, int32_t lo_block, int32_t hi_block,
                         const bf1_route_cfg *cfg /* host */, const int32_t *needed_blocks_dev,
                         int32_t num_needed, const bf1_route *out /* host struct, device arrays */,
                         int32_t *cu_seqlens_out_dev /* [2] */, void *stream);

/* The same two plans for a shard that owns every `stride`-th block: first_block, first_block + stride, ...,
 * num_blocks of them (rank r of R ranks: first_block = r, stride = R).  The route is block aligned and data
 * independent (Section 3.1) and its long edges are powers of two (Eq. 1), so with a power-of-two stride the dyadic
 * predecessors j - 2^k with 2^k >= stride of an owned block are owned as well: a rank is sent little more than the
 * window in front of each of its blocks and block 0 (about two blocks per own block, whatever its rank), and all
 * ranks hold lists of the same lengths -- where contiguous shards leave the first rank with the short lists and
 * send the last one most of the sequence.  The local key/value tensor is laid out as before, [the needed blocks in
 * ascending global order | the own blocks in ascending order]; a list is re-indexed entry by entry, so its local
 * indices end in the query block itself but need not ascend (the attention kernel does not require it). */
int bf1_shard_needed_blocks_strided(int64_t n_tokens, const bf1_route_cfg *cfg /* host */, int32_t first_block,
                                    int32_t stride, int32_t num_blocks, int32_t *blocks_out /* host */,
                                    int32_t capacity, int32_t *count_out /* host */);
int bf1_plan_route_shard_strided(int64_t n_tokens, int32_t first_block, int32_t stride, int32_t num_blocks,
                                 const bf1_route_cfg *cfg /* host */, const int32_t *needed_blocks_dev,
                                 int32_t num_needed, const bf1_route *out /* host struct, device arrays */,
                                 int32_t *cu_seqlens_out_dev, void *stream);


/* Message for the last non-OK status returned on the calling thread ("" if none). */
const char *bf1_last_error(void);

/* Library version, for the binding's sanity check. */
int bf1_version(void);

#ifdef __cplusplus
}
#endif
#endif /* BF1_H_ */

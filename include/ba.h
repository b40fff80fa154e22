/*
 * ba.h -- C ABI of the Block-attention prefilling hot path for NVIDIA B200 (sm_100a).
 *
 * The library implements, as CUDA kernels, the three data-parallel steps of
 * Block-attention inference (arXiv 2409.15355):
 *
 *   (a) position re-encoding of cached per-block keys         Section 2.3, Eq. 1-3
 *   (b) the final block attending every cached block + itself Section 2.5, step 3
 *   (c) block-diagonal prefill of all blocks in one launch    Section 1; Section 2.4
 *
 * plus the integer tables that describe a ragged prompt (Section 2.2, 2.5) and a
 * flag that switches the same entry points to ordinary full causal attention
 * (Section 3: the fine-tuned model runs under either mask).
 *
 * Conventions
 * -----------
 * - Tensors are DEVICE pointers owned by the caller, row-major
 *   [tokens, heads, head_dim], bfloat16 unless stated, base address 16-byte
 *   aligned, tokens packed without padding.
 * - Three packings of a batch of prompts are used.  "prompt packing": every
 *   block of every sequence in prompt order (n_tokens rows).  "cache packing":
 *   only the non-final blocks, in the same order.  "final packing": only the
 *   final block of every sequence, in sequence order.
 * - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is
 *   the default stream).  Argument and launch errors are returned at once.
 *   Problems only the device can see (inconsistent tables, a bounded wait that
 *   ran out) are recorded in a status word read by ba_last_device_status().
 * - Nothing is allocated after ba_create(); a workspace that is too small for a
 *   call yields BA_ERR_WORKSPACE.  Calls on one context share its workspace, so
 *   they must be ordered on the device (one stream, or events between streams);
 *   the one exception is ba_reencode_k with the cache_delta array of the
 *   context's current tables, which uses no workspace and may run on another
 *   stream beside an attention call that does not read or write its tensors.
 *   All calls on a context come from one host thread at a time.
 * - Every call that takes a context makes that context's device the calling
 *   thread's current CUDA device (cudaSetDevice) and leaves it current on return;
 *   ba_reencode_k_noalloc does the same with its `device` argument.
 * - No C++ exceptions cross this boundary.  There is no CPU fallback: on a
 *   machine without a usable sm_100 device ba_create() fails.
 */
#ifndef BA_H_
#define BA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct ba_ctx ba_ctx; /* opaque */

typedef enum {
  BA_OK = 0,
  BA_ERR_INVALID_ARG = 1, /* null / misaligned pointer, bad enum, inconsistent lengths */
  BA_ERR_SHAPE = 2,       /* sizes that do not fit together */
  BA_ERR_UNSUPPORTED = 3, /* head_dim not in {64,128}, n_q_heads % n_kv_heads != 0, ... */
  BA_ERR_WORKSPACE = 4,   /* workspace given to ba_create too small for this call */
  BA_ERR_CUDA = 5,        /* a CUDA runtime/driver call failed */
  BA_ERR_TIMEOUT = 6      /* a bounded device-side wait expired */
} ba_status;

typedef enum { BA_MODE_BLOCK = 0, BA_MODE_FULL = 1 } ba_mode;

/* Which coordinates form rotary pair m.  Eq. 1 draws 2x2 blocks on the diagonal,
 * i.e. pairs (2m, 2m+1): BA_ROPE_ADJACENT.  BA_ROPE_HALF pairs (m, m + head_dim/2). */
typedef enum { BA_ROPE_ADJACENT = 0, BA_ROPE_HALF = 1 } ba_rope_layout;

typedef enum { BA_OUT_BF16 = 0, BA_OUT_F32 = 1 } ba_out_dtype;

typedef struct {
  int32_t n_q_heads;
  int32_t n_kv_heads;    /* query head h reads KV head h / (n_q_heads / n_kv_heads) */
  int32_t head_dim;      /* 64 or 128 */
  int32_t rope_layout;   /* ba_rope_layout */
  double rope_theta;     /* base of theta_m = base^(-2m/head_dim) */
  float softmax_scale;   /* 0 selects 1/sqrt(head_dim) */
  int32_t reserved;
} ba_config;

/*
 * Tables of a ragged batch, produced by ba_segment().  The struct lives on the
 * host; every pointer is a DEVICE pointer into the caller's table buffer.
 * B = n_blocks, T = n_tokens, Bc = n_blocks - batch (each sequence has exactly
 * one final block).
 */
typedef struct {
  int32_t batch, n_blocks, n_tokens, n_cached_blocks;
  int32_t mode;            /* ba_mode the tables were built for */
  int32_t q_tile_tokens;   /* tokens per query tile of the attention kernels */
  int32_t n_prompt_items;  /* work items of ba_block_prefill / ba_final_attend for these tables when the */
  int32_t n_final_items;   /* lengths were host arrays (exact launch size); 0 when they were on the device */
  /* 128-key tiles the work items of ba_final_attend see, when the lengths were host arrays (else 0):
   * sum, minimum and maximum over the items, [0..2] with the cached keys of a sequence packed in one run,
   * [3..5] with every cached block starting a tile of its own (pools, fused path).  Used to balance the launch. */
  int32_t final_key_tiles[6];
  /* per sequence, [batch + 1] */
  int32_t *cu_seq;         /* first row of the sequence, prompt packing */
  int32_t *cu_cache_seq;   /* first row of the sequence, cache packing */
  int32_t *cu_final_seq;   /* first row of the sequence, final packing */
  int32_t *cu_seq_block;   /* index of the sequence's first block */
  /* per block */
  int32_t *cu_block;       /* [B+1] first row of the block, prompt packing */
  int32_t *block_delta;    /* [B] prompt position of the block's first token = re-encoding delta */
  int32_t *block_seq;      /* [B] sequence the block belongs to */
  int32_t *block_kv_begin; /* [B] first key row (prompt packing) rows of this block may see */
  int32_t *block_part_off; /* [B] first row of the block in cache packing (non-final) or final packing (final) */
  uint8_t *block_is_final; /* [B] */
  /* the non-final blocks, in order: the arguments of ba_reencode_k */
  int32_t *cache_block;    /* [Bc] index of the block in the prompt */
  int32_t *cache_cu;       /* [Bc+1] first row, cache packing */
  int32_t *cache_delta;    /* [Bc] */
  /* per token, [T] */
  int32_t *tok_block;
  int32_t *tok_pos;        /* position in the prompt (0-based within its sequence) */
  int32_t *tok_pos_local;  /* position inside its block = position it has in the cache */
  /* query-tile tables used by the attention kernels (not part of the bit-exact contract) */
  int32_t *cu_qtile;       /* [B+1] */
  int32_t *cu_ftile;       /* [batch+1] */
  int32_t *cache_tile_cu;  /* [Bc+1] prefix sum of 128-key tiles per cached block (a tile never spans two blocks) */
  int32_t *cu_ktile;       /* [B+1] prefix sum of 128-key tiles per block, every block (backward pass) */
  int32_t *totals;         /* [8]: cached tokens, final tokens, q tiles, final tiles, ..., [7] = validity word */
  /* rotation of every cached block, used by ba_final_attend_fused: (cos, sin)(cache_delta[c] * theta_m),
   * fp32 from fp64 angles, [Bc][head_dim / 2][2] */
  float *cache_rope;
} ba_segments;

/* Create a context on CUDA device `device` and allocate `workspace_bytes` of
 * scratch there (rotation tables, split-KV partial results).  Fails with
 * BA_ERR_UNSUPPORTED for shapes outside the supported set and with BA_ERR_CUDA
 * when the device is missing or is not compute capability 10.x. */
ba_status ba_create(ba_ctx **ctx, const ba_config *cfg, int device, size_t workspace_bytes);
ba_status ba_destroy(ba_ctx *ctx);
const char *ba_status_string(ba_status s);

/* Workspace ba_create() should be given so that calls of at most these sizes fit: max_blocks cached
 * blocks per re-encoding call, max_q_rows query rows per attention call (split-KV partial results are
 * only used for short query sides) and per backward call (its dO . O buffer). */
ba_status ba_workspace_bytes(const ba_config *cfg, int32_t max_blocks, int32_t max_q_rows, size_t *bytes);

/* Synchronises the context's device and returns (then clears) the first
 * problem a kernel recorded since the last call: BA_OK, BA_ERR_INVALID_ARG
 * (tables inconsistent with the lengths given; a gather index outside its source;
 * a rotation table that no longer belongs to the tables it was stored with),
 * BA_ERR_SHAPE (the tables describe more query rows than the tensors passed to an
 * attention call hold: the surplus rows are not written) or BA_ERR_TIMEOUT. */
ba_status ba_last_device_status(ba_ctx *ctx);

/* Diagnostic (no counterpart in the paper): launches one CTA that waits, with the library's
 * bounded wait, on a barrier nothing completes.  After about a second the wait gives up and
 * ba_last_device_status() returns BA_ERR_TIMEOUT; the device stays usable.  Lets a deployment
 * check the expiry path of the attention kernels without provoking a fault. */
ba_status ba_selftest_wait_expiry(ba_ctx *ctx, void *stream);

/* Number of this library's kernels launched through `ctx` so far. */
int64_t ba_launch_count(const ba_ctx *ctx);

/* Diagnostic: how the last attention launch through `ctx` was laid out.  out[0] = CTAs, out[1] = partial
 * results per row that a second kernel merges (1: none), out[2] = CTAs that each took the tail of one work
 * item in a balanced launch (0: not balanced), out[3] = key tiles of such a tail. */
ba_status ba_last_attend_shape(const ba_ctx *ctx, int32_t out[4]);

/* Diagnostic, no device needed: the planning step of ba_final_attend as a function of its inputs.  n_sms SMs,
 * n_pairs work items per head chunk (ba_segments.n_final_items), n_head_chunks head chunks, avg_key_tiles 128-key
 * tiles of an average item, key_tiles = {sum, minimum, maximum} of the key tiles over the n_pairs items (zeros:
 * unknown), max_partials = the most partial results per row the workspace has room for.  out[0] = partial results
 * per row (1: no split), out[1] = CTAs that take the tail of one item each (0: equal splits), out[2] = key tiles
 * of such a tail. */
ba_status ba_plan_final_attend(int32_t n_sms, int32_t n_pairs, int32_t n_head_chunks, int32_t avg_key_tiles,
                               const int32_t key_tiles[3], int32_t max_partials, int32_t out[3]);

/* Bytes of the table buffer ba_segment() needs for these sizes. */
ba_status ba_segments_bytes(int32_t batch, int32_t n_blocks, int32_t n_tokens, size_t *bytes);

/*
 * Section 2.2 / 2.5: tables of a ragged batch from its block lengths.
 *   block_lens  [n_blocks]  length of every block, prompt order; host or device memory
 *   seq_nblocks [batch]     blocks per sequence (its last block is the final block); host or device
 *   n_tokens                sum of block_lens (the caller sized its tensors with it)
 *   mode                    BA_MODE_FULL makes every row see its whole sequence prefix
 *                           (block_kv_begin = cu_seq); all other tables are unchanged
 *   table_buf               device buffer of at least ba_segments_bytes() bytes, 16-byte aligned
 *   out                     host struct, filled with pointers into table_buf
 * With host arrays the lengths are checked before launching (BA_ERR_INVALID_ARG
 * for a length < 1 or sums that do not match); with device arrays the same
 * check runs on the device and is reported by ba_last_device_status().
 */
ba_status ba_segment(ba_ctx *ctx, const int32_t *block_lens, const int32_t *seq_nblocks,
                     int32_t batch, int32_t n_blocks, int32_t n_tokens, ba_mode mode,
                     void *table_buf, size_t table_bytes, ba_segments *out, void *stream);

/*
 * Section 2.3, Eq. 1-3: rotate cached keys from their cache positions to their
 * positions in the new prompt.  For block c (0 <= c < n_blocks) and row t of it,
 * every KV head and rotary pair m:
 *     (x, y) <- (x cos(a) - y sin(a), x sin(a) + y cos(a)),  a = delta[c] * theta_m.
 * A positive delta is Eq. 3 applied after Eq. 2 (the two collapse into one
 * rotation by the difference, as Section 2.3 notes); a negative delta is Eq. 2
 * (back to position zero, e.g. to fill the cache after a cold prefill); delta 0
 * copies bit-exactly.
 *   k_src    bf16 [n_src_rows, n_kv_heads, head_dim]; block c is read from row src_off[c], or
 *            from row cu[c] when src_off is NULL.  A source row outside [0, n_src_rows) is
 *            skipped and reported through ba_last_device_status() as BA_ERR_INVALID_ARG.
 *   k_dst    bf16 [n_rows, n_kv_heads, head_dim]; block c is written to rows cu[c]..cu[c+1]-1.
 *            May equal k_src when src_off is NULL (in place).
 *   cu       device int32 [n_blocks+1], delta device int32 [n_blocks], src_off device int32 or NULL
 *   n_rows   rows of k_dst (>= cu[n_blocks]); rows beyond cu[n_blocks] are not touched
 * Uses n_blocks * head_dim * 4 bytes of workspace for the angle table.  When `delta` is the
 * cache_delta array of the tables this context's last ba_segment() built (and n_blocks their
 * cached-block count), the rotation table built with those tables is used instead and no table is
 * computed; those tables must then still be alive and unchanged.  (ba_segment() stamps its tables;
 * if the buffer was rebuilt or overwritten in the meantime the call rotates nothing and
 * ba_last_device_status() reports BA_ERR_INVALID_ARG.)
 */
ba_status ba_reencode_k(ba_ctx *ctx, const void *k_src, const int32_t *src_off, int32_t n_src_rows,
                        void *k_dst, const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                        int32_t n_rows, void *stream);

/*
 * Section 2.5, across layers: the cached keys of every layer are known the moment the cache is
 * hit, so the re-encoding of layer l+1 need not wait for the attention of layer l.
 * ba_reencode_k_deferred queues the job described by its arguments (the same as ba_reencode_k):
 * the angle table is computed at once on `stream`, the rotation itself is carried out by otherwise
 * idle warps of the NEXT ba_final_attend / ba_block_prefill launched through this context, in the
 * background of that kernel, and is complete when that kernel completes (stream order, as usual).
 * The job must not touch the tensors that attention call reads or writes.  One job can be queued
 * per context: queuing another, ba_flush() or ba_destroy() run a still-queued job as an ordinary
 * stand-alone launch.  Results are bit-identical to ba_reencode_k.  The queued job's arguments
 * (device pointers) must stay valid until it has run.
 */
ba_status ba_reencode_k_deferred(ba_ctx *ctx, const void *k_src, const int32_t *src_off, int32_t n_src_rows,
                                 void *k_dst, const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                                 int32_t n_rows, void *stream);
/* Runs a queued re-encoding job now, on `stream`; does nothing when none is queued. */
ba_status ba_flush(ba_ctx *ctx, void *stream);

/*
 * ba_reencode_k_noalloc -- the same re-encoding as ba_reencode_k for callers that
 * must not allocate device memory.  (The paper has no counterpart to this entry
 * point; it exists for integration reasons only.)
 *
 * Who needs it: a serving engine that hands all free device memory to its own
 * pool at start-up (a later cudaMalloc then fails or eats into the pool's
 * head-room), and code on a latency-critical path that cannot afford the
 * device-wide synchronisation cudaMalloc/cudaFree imply.  Such callers cannot
 * use ba_create(), which allocates the workspace the angle table lives in.
 *
 * This call needs no context.  The angle table is kept in a fixed array built
 * into the library image: BA_NOALLOC_MAX_BLOCKS * 64 (cos, sin) pairs = 2 MiB
 * that every GPU which loads the library holds until the process exits.  The
 * call itself performs no cudaMalloc/cudaFree and uses no allocating library
 * routine.
 *
 *   cfg, device    as for ba_create (head_dim, n_kv_heads, rope_theta, rope_layout are used); the
 *                  device must exist (BA_ERR_CUDA otherwise), becomes the thread's current device,
 *                  and gets a CUDA context if it had none
 *   status_word    device int32 owned by the caller, or NULL.  A source row out of range is
 *                  skipped and BA_ERR_INVALID_ARG is stored there if the word is still 0
 *                  (clear it yourself); with NULL such rows are skipped silently.
 *   other arguments exactly as for ba_reencode_k
 *
 * n_blocks > BA_NOALLOC_MAX_BLOCKS is rejected with BA_ERR_WORKSPACE before anything runs.
 * The first call on a device looks up the device address of the built-in array;
 * make that first call outside any stream capture.  All calls on a device share
 * the one array, which keeps the previous call's contents (every entry a call
 * reads is rewritten by that call first, so nothing needs clearing): two calls
 * whose kernels may overlap on the GPU -- different streams, no ordering between
 * them -- race on it and must be ordered by the caller.
 */
#define BA_NOALLOC_MAX_BLOCKS 4096
ba_status ba_reencode_k_noalloc(const ba_config *cfg, int device, const void *k_src,
                                const int32_t *src_off, int32_t n_src_rows, void *k_dst,
                                const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                                int32_t n_rows, int32_t *status_word, void *stream);

/*
 * Section 1 / Section 2.4: attention of a packed ragged batch under the
 * Block-attention mask, all blocks in one launch.  Row i of block b sees key
 * rows block_kv_begin[b] .. i (prompt packing).  q [T, n_q_heads, head_dim],
 * k, v [T, n_kv_heads, head_dim] bf16 with RoPE already applied at tok_pos;
 * o [T, n_q_heads, head_dim] bf16 or fp32; lse fp32 [T, n_q_heads] or NULL
 * (natural-log softmax denominator).  `mode` must equal seg->mode.
 */
ba_status ba_block_prefill(ba_ctx *ctx, const void *q, const void *k, const void *v, void *o,
                           float *lse, const ba_segments *seg, ba_mode mode,
                           ba_out_dtype out_dtype, void *stream);

/*
 * Section 2.5, step 3: the final block of every sequence attends that
 * sequence's cached blocks and itself (causally).
 *   q_f, k_f, v_f   final packing, [n_final_rows, heads, head_dim] bf16, RoPE at prompt positions
 *   k_cache         bf16 keys of the cached blocks at their PROMPT positions (the output
 *                   of ba_reencode_k), cache packing, n_cache_rows rows
 *   v_cache         bf16 values of the cached blocks: cache packing when v_src_off is NULL,
 *                   else a pool of n_v_rows rows in which cached block c starts at v_src_off[c]
 *   o               final packing, [n_final_rows, n_q_heads, head_dim]; lse [n_final_rows, n_q_heads] or NULL
 * The mode flag does not change the result (final rows see the same keys under
 * both masks) but must equal seg->mode.
 */
ba_status ba_final_attend(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                          int32_t n_final_rows, const void *k_cache, const void *v_cache,
                          int32_t n_cache_rows, const int32_t *v_src_off, int32_t n_v_rows,
                          void *o, float *lse, const ba_segments *seg, ba_mode mode,
                          ba_out_dtype out_dtype, void *stream);

/*
 * Section 2.5, steps 2 and 3 in one launch: the final block of every sequence attends that
 * sequence's cached blocks and itself, with the cached keys still at their CACHE-TIME positions
 * (token t of a block rotated to position t, as Section 2.3 stores them).  The position
 * re-encoding of Eq. 3 after Eq. 2 -- one rotation by the block's delta -- is applied to the
 * other side of the dot product: (R(p) q) . (R(delta + t) k) = (R(-delta) R(p) q) . (R(t) k),
 * so the query tiles are rotated once per cached block on chip and the cached keys are neither
 * rewritten nor read twice.  The result equals ba_reencode_k followed by ba_final_attend up to
 * the rounding of the rotated operand to bf16 (queries here, keys there).  The re-encoded keys
 * themselves -- what the rest of generation reads -- are written as a side output when k_out is
 * given: the call then also runs the re-encoding kernel, on a stream of the context's own beside the
 * attention launch (which leaves SMs idle in its last wave), and joins it back into `stream`; k_out is
 * bit-identical to ba_reencode_k's output and complete, in stream order, when the call is.
 *   q_f, k_f, v_f   as for ba_final_attend
 *   k_src, v_src    bf16 [n_src_rows, n_kv_heads, head_dim]: cached block c (cache order, as in
 *                   seg->cache_cu) occupies rows src_off[c] .. src_off[c] + length - 1 of both, or
 *                   rows cache_cu[c] .. when src_off is NULL (cache packing)
 *   n_cache_rows    total cached rows of the batch (= cache_cu[Bc])
 *   k_out           NULL, or bf16 [n_cache_rows, n_kv_heads, head_dim] (cache packing), not k_src
 *   seg             tables of ba_segment(); its cache_rope table holds the rotations
 * A queued ba_reencode_k_deferred job is run as a stand-alone launch first.
 */
ba_status ba_final_attend_fused(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                                int32_t n_final_rows, const void *k_src, const void *v_src,
                                int32_t n_src_rows, const int32_t *src_off, int32_t n_cache_rows,
                                void *k_out, void *o, float *lse, const ba_segments *seg, ba_mode mode,
                                ba_out_dtype out_dtype, void *stream);

/*
 * Section 2.4 (block fine-tune): backward pass of ba_block_prefill.  Block fine-tuning trains the
 * model with the Block-attention mask in place of the lower-triangular one, so the gradients flow
 * through the same masked softmax: with P = softmax(scale Q K^T + mask), O = P V,
 *     dV = P^T dO,   dS = P * (dO V^T - rowsum(dO * O)),   dQ = scale dS K,   dK = scale dS^T Q,
 * dK and dV summed over the query heads that share a KV head.  P is recomputed from `lse`.
 *   q, k, v, seg, mode   exactly what the forward call was given
 *   o                    bf16 [T, n_q_heads, head_dim]: the forward output (BA_OUT_BF16)
 *   lse                  fp32 [T, n_q_heads]: the forward call's log-sum-exp (required)
 *   d_o                  bf16 [T, n_q_heads, head_dim]: gradient of the loss with respect to o
 *   dq                   [T, n_q_heads, head_dim];  dk, dv  [T, n_kv_heads, head_dim]; bf16 or fp32
 * Uses T * n_q_heads * 4 bytes of workspace (BA_ERR_WORKSPACE when the context has less).  No
 * atomics: results are run-to-run identical.
 */
ba_status ba_block_prefill_bwd(ba_ctx *ctx, const void *q, const void *k, const void *v, const void *o,
                               const float *lse, const void *d_o, void *dq, void *dk, void *dv,
                               const ba_segments *seg, ba_mode mode, ba_out_dtype grad_dtype, void *stream);

/*
 * Paged KV pool (Section 2.3: what the cache holds; Section 2.5 step 1: the cache look-up).  A serving
 * cache rarely keeps a passage in one piece: it hands out fixed-size pages.  Here the cached keys and
 * values of all blocks live in pool tensors [n_pages * page_rows, n_kv_heads, head_dim] (one for K, one
 * for V, same paging), page `g` being rows g * page_rows .. (g + 1) * page_rows - 1.  Cached block c
 * (cache order, as in seg->cache_cu) owns the pages page_idx[page_cu[c]] .. page_idx[page_cu[c+1] - 1],
 * in that order: row t of the block is row t % page_rows of its page number t / page_rows; a block
 * of length L has ceil(L / page_rows) pages and the rest of its last page is not part of it.  Those
 * unused rows must hold finite values (a pool that started out zeroed, or stale keys and values):
 * they are masked, but a tensor-core product of zero with a NaN bit pattern would still be NaN.
 *   page_rows   a power of two, 16 .. 65536
 *   page_cu     device int32 [n_blocks + 1], page_idx device int32 [page_cu[n_blocks]]
 * A page number outside [0, n_pages) is never read: ba_reencode_k_paged skips the row and reports
 * BA_ERR_INVALID_ARG through ba_last_device_status(); the attention calls read zeros in its place.
 */
typedef struct {
  int32_t page_rows;
  int32_t n_pages;
  const int32_t *page_cu;
  const int32_t *page_idx;
} ba_page_table;

/* ba_reencode_k with the cached keys gathered from a paged pool (Eq. 1-3 as there); k_dst in cache
 * packing, cu / delta / n_blocks / n_rows as for ba_reencode_k. */
ba_status ba_reencode_k_paged(ba_ctx *ctx, const void *k_pool, const ba_page_table *pages, void *k_dst,
                              const int32_t *cu, const int32_t *delta, int32_t n_blocks, int32_t n_rows,
                              void *stream);

/* ba_final_attend (Section 2.5 step 3) with the cached VALUES read in place from a paged pool; the
 * re-encoded keys k_cache are in cache packing (the output of ba_reencode_k_paged).  A key tile of the
 * kernel never spans two pages: it is assembled from one copy per page. */
ba_status ba_final_attend_paged(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                                int32_t n_final_rows, const void *k_cache, int32_t n_cache_rows,
                                const void *v_pool, const ba_page_table *pages, void *o, float *lse,
                                const ba_segments *seg, ba_mode mode, ba_out_dtype out_dtype, void *stream);

/* ba_final_attend_fused (Section 2.5 steps 2-3 in one launch) with cached keys (at cache-time positions)
 * and values both read in place from paged pools that share one page table; k_out as there. */
ba_status ba_final_attend_fused_paged(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                                      int32_t n_final_rows, const void *k_pool, const void *v_pool,
                                      const ba_page_table *pages, int32_t n_cache_rows, void *k_out,
                                      void *o, float *lse, const ba_segments *seg, ba_mode mode,
                                      ba_out_dtype out_dtype, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* BA_H_ */

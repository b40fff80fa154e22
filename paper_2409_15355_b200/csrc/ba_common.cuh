// Internal declarations shared by the translation units of the library.
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "ba.h"

// A failed runtime call also leaves its code in the runtime's per-thread "last error" slot; it is
// cleared here so that a later, healthy launch does not trip over it.
#define BA_CUDA_TRY(expr)                                              \
  do {                                                                 \
    cudaError_t _e = (expr);                                           \
    if (_e != cudaSuccess) { cudaGetLastError(); return BA_ERR_CUDA; } \
  } while (0)

// Value of ba_segments::totals[7] once ba_segment's kernel has found the lengths consistent.
#define BA_TABLES_VALID 0x600D

// One re-encoding job: block c of `n_blocks` is read from row src_off[c] (or cu[c]) of `src`,
// rotated by delta[c] with the (cos, sin) pairs in `table`, and written to rows cu[c].. of `dst`.
struct ba_reencode_job {
  const uint4 *src;
  uint4 *dst;
  const int32_t *src_off;
  const int32_t *cu;
  const int32_t *delta;
  const float2 *table;      // [n_blocks][head_dim / 2] (cos, sin)
  int32_t n_src_rows, n_blocks, n_rows;
  int32_t head_dim, row_vecs /* uint4 per row */, layout;
  // non-null: `table` is the rotation table ba_segment() stored with its tables; *gen must still hold
  // gen_expected (the stamp that call wrote), else the tables were rebuilt or overwritten since and
  // the job reports BA_ERR_INVALID_ARG instead of rotating with a foreign table
  const int32_t *gen;
  int32_t gen_expected;
  // non-null: the source is a paged pool -- block c owns pages page_idx[page_cu[c] .. page_cu[c+1]) of
  // 1 << page_lg rows each (src_off is ignored)
  const int32_t *page_cu, *page_idx;
  int32_t page_lg;
};

// Source row of row `t` (0-based inside its block) of a job's block `c`; negative when the page number is bad.
__device__ __forceinline__ long long ba_job_source_row(const ba_reencode_job &job, int c, int c_begin, int t) {
  if (job.page_cu) {
    const int page = __ldg(job.page_idx + __ldg(job.page_cu + c) + (t >> job.page_lg));
    if (page < 0) return -1;
    return ((long long)page << job.page_lg) + (t & ((1 << job.page_lg) - 1));
  }
  return (job.src_off ? (long long)__ldg(job.src_off + c) : (long long)c_begin) + t;
}

// Context: configuration, workspace and the device status word.
struct ba_ctx {
  ba_config cfg;
  int device;
  int sm_count;
  float scale;              // softmax scale actually used
  void *workspace;          // device
  size_t workspace_bytes;
  int32_t *dev_status;      // device word: first non-zero ba_status recorded by a kernel
  int64_t launches;
  int32_t last_attend[4];          // layout of the last attention launch: CTAs, partial slots, balanced tails, tail tiles
  // a re-encoding job queued by ba_reencode_k_deferred: carried along by the next attention
  // launch (or run by ba_flush); its angle table sits at the very end of the workspace
  ba_reencode_job pending;
  int has_pending;
  size_t pending_table_bytes;
  cudaStream_t pending_stream;
  // rotation table of the cached blocks built by the last ba_segment (in the caller's table buffer):
  // a re-encoding call whose delta array is that table's cache_delta reuses it instead of rebuilding it
  const int32_t *seg_delta;
  const float2 *seg_rope;
  int32_t seg_rope_blocks;
  const int32_t *seg_gen;   // device word the same ba_segment stamped with seg_gen_value (totals[6])
  int32_t seg_gen_value;
  int32_t seg_counter;      // ba_segment calls so far on this context
  // tensor maps of recently used tensors (attention launches re-use a handful of buffers)
  struct ba_map_cache *maps;
  // side stream of the fused call's key write-back (forked from and joined to the caller's stream by events)
  cudaStream_t side_stream;
  cudaEvent_t ev_fork, ev_join;
};

static inline size_t ba_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Workspace layout: [0, 64 KiB) staging of host-side length arrays (ba_segment);
// [64 KiB, ...) per-call scratch: split-KV partial results (attention) or, at the very end
// of the workspace, the angle table (re-encode).  Calls on one context are stream-ordered,
// so the regions may be reused from call to call.
static inline size_t ba_scratch_offset(const ba_ctx *) { return 64 * 1024; }

// How ba_final_attend divides the key tiles of its work items among CTAs (pure host arithmetic, also reachable
// through ba_plan_final_attend).  Inputs: SMs; work items (query tile pairs x head chunks); pairs and head chunks;
// key tiles of an average item; sum / minimum / maximum of the key tiles over the pairs when known (else zeros);
// the most partial results per row the workspace has room for.
//  * Equal splits: n_splits entries per item, the count that minimises waves x (tiles per entry + 3), the 3
//    standing for an entry's start-up and write-out.
//  * Balanced launch (item sizes known, fewer items than SMs, every item longer than an SM's share of the tiles):
//    one CTA per item takes the item's last `len` key tiles, the remaining CTAs share the tiles in front of those
//    in equal runs.  `len` starts at the even share and grows until the CTAs that work on several pieces (each
//    with its own start-up and write-out, plus 1 for their table) are no longer the slower ones.  Taken when the
//    same cost model puts it ahead of equal splits; n_splits is then the number of partial results per row.
constexpr int kBalMaxPairs = 120;        // the balanced launch keeps a prefix table of this many pairs in shared memory
struct ba_split_plan { int n_splits, balanced, bal_len; };
static inline ba_split_plan ba_plan_splits(int sm_count, long long items, int n_pairs, int n_chunks, long long avg_tiles,
                                           const int32_t *key_tiles, int cap) {
  ba_split_plan plan = {1, 0, 0};
  if (items >= 2LL * sm_count || cap < 1) return plan;
  long long best = -1;
  for (int ns = 1; ns <= cap && ns <= avg_tiles; ++ns) {
    const long long waves = (items * ns + sm_count - 1) / sm_count;
    const long long cost = waves * ((avg_tiles + ns - 1) / ns + 3);
    if (best < 0 || cost < best) { best = cost; plan.n_splits = ns; }
  }
  const long long n_main = (long long)n_pairs * n_chunks;
  const long long n_front = sm_count - n_main;
  if (key_tiles[0] > 0 && n_main > 0 && n_front > 0 && n_pairs <= kBalMaxPairs) {
    const long long total = (long long)key_tiles[0] * n_chunks, n_min = key_tiles[1], n_max = key_tiles[2];
    for (long long len = (total + sm_count - 1) / sm_count; len <= n_min; ++len) {
      const long long front = total - n_main * len;
      if (front <= 0) break;
      const long long run = (front + n_front - 1) / n_front, run_min = front / n_front;
      if (run_min < 1) break;
      const long long piece = (front + n_main - 1) / n_main;          // average front tiles of an item
      const long long cost_front = run + 3 * ((run + piece - 1) / piece + 1) + 1;
      if (cost_front > len + 3) continue;
      const long long slots = 1 + (n_max - len + run_min - 1) / run_min + 1;
      if (len + 3 < best && slots <= cap) { plan.balanced = (int)n_main; plan.bal_len = (int)len; plan.n_splits = (int)slots; }
      break;
    }
  }
  return plan;
}

// Records the first device-side problem; later ones are dropped.
__device__ __forceinline__ void ba_record_status(int32_t *status, int32_t code) {
  atomicCAS(status, 0, code);
}

// Entry points implemented in the individual .cu files.
ba_status ba_segment_launch(ba_ctx *ctx, const int32_t *d_block_lens, const int32_t *d_seq_nblocks,
                            int32_t batch, int32_t n_blocks, int32_t n_tokens, int mode, int32_t gen,
                            const ba_segments *seg, cudaStream_t stream);

// Re-encoding in two steps: angle table, then the rotation itself.
ba_status ba_reencode_table_launch(ba_ctx *ctx, const int32_t *delta, int32_t n_blocks, float2 *table,
                                   cudaStream_t stream);
ba_status ba_reencode_main_launch(ba_ctx *ctx, const ba_reencode_job &job, cudaStream_t stream);
ba_status ba_reencode_launch(ba_ctx *ctx, const void *k_src, const int32_t *src_off,
                             int32_t n_src_rows, void *k_dst, const int32_t *cu,
                             const int32_t *delta, int32_t n_blocks, int32_t n_rows, float2 *table,
                             cudaStream_t stream);
ba_reencode_job ba_make_reencode_job(const ba_ctx *ctx, const void *k_src, const int32_t *src_off,
                                     int32_t n_src_rows, void *k_dst, const int32_t *cu, const int32_t *delta,
                                     int32_t n_blocks, int32_t n_rows, const float2 *table);
// Runs a pending deferred job as a stand-alone launch (no-op when nothing is pending).
ba_status ba_flush_pending(ba_ctx *ctx, cudaStream_t stream);

struct ba_attend_args {
  // queries / outputs: rows of the q packing (prompt packing for prefill, final packing for final attend)
  const __nv_bfloat16 *q;
  void *o;
  float *lse;
  int32_t n_q_rows;
  int out_f32;
  // primary keys/values: same packing as q (prefill: the whole prompt; final attend: the final blocks)
  const __nv_bfloat16 *k, *v;
  int32_t n_kv_rows;
  // cached keys/values (final attend only)
  const __nv_bfloat16 *k_cache, *v_cache;
  int32_t n_cache_rows, n_v_rows;
  const int32_t *v_src_off;
  // fused warm path: k_cache holds the cached keys at cache-time positions (n_k_rows rows; block c
  // at row k_src_off[c], or at its packed offset when k_src_off is null)
  int fused;
  const int32_t *k_src_off;
  int32_t n_k_rows;
  void *k_out;     // fused warm path: non-null -> the re-encoded keys are also written here (cache packing)
  // paged pool (page_rows > 0): the cached values -- and on the fused path the cached keys -- are read
  // through a page table instead of v_src_off / k_src_off
  int32_t page_rows;
  const int32_t *page_cu, *page_idx;
  int final_only;  // 1: ba_final_attend, 0: ba_block_prefill
};

ba_status ba_attend_launch(ba_ctx *ctx, const ba_attend_args &a, const ba_segments *seg,
                           cudaStream_t stream);

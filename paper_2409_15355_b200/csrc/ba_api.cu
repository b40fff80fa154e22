// Host side of the C ABI: argument checks, table-buffer layout, workspace
// bookkeeping and dispatch to the kernels.  No kernel code lives here.
#include <algorithm>
#include <new>
#include <string.h>

#include "ba_common.cuh"

ba_status ba_attend_sm100_launch(ba_ctx *ctx, const ba_attend_args &a, const ba_segments *seg,
                                 cudaStream_t stream);
ba_status ba_attend_sm100_setup(ba_ctx *ctx);
ba_status ba_bwd_sm100_setup(ba_ctx *ctx);
ba_status ba_bwd_sm100_launch(ba_ctx *ctx, const void *q, const void *k, const void *v, const void *o,
                              const float *lse, const void *d_o, void *dq, void *dk, void *dv, int out_f32,
                              const ba_segments *seg, int mode, cudaStream_t stream);
void ba_attend_sm100_teardown(ba_ctx *ctx);
int ba_heads_per_tile(const ba_config &c);

namespace {

bool aligned16(const void *p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Is `p` ordinary host memory (to be staged), as opposed to device-visible memory?
bool is_host_pointer(const void *p) {
  cudaPointerAttributes at;
  cudaError_t e = cudaPointerGetAttributes(&at, p);
  if (e != cudaSuccess) { cudaGetLastError(); return true; }
  return at.type == cudaMemoryTypeUnregistered || at.type == cudaMemoryTypeHost;
}

ba_status check_config(const ba_config *c) {
  if (!c) return BA_ERR_INVALID_ARG;
  if (c->head_dim != 64 && c->head_dim != 128) return BA_ERR_UNSUPPORTED;
  if (c->n_q_heads < 1 || c->n_kv_heads < 1 || c->n_q_heads % c->n_kv_heads) return BA_ERR_UNSUPPORTED;
  if (c->rope_layout != BA_ROPE_ADJACENT && c->rope_layout != BA_ROPE_HALF) return BA_ERR_INVALID_ARG;
  if (!(c->rope_theta > 1.0)) return BA_ERR_INVALID_ARG;
  if (c->softmax_scale < 0.f) return BA_ERR_INVALID_ARG;
  return BA_OK;
}

// Tokens per work item of the tensor-core attention kernel: two query tiles of
// 128 rows, each row one (token, head) of the heads packed into a tile.
int q_tile_tokens(const ba_config &c) { return 2 * 128 / ba_heads_per_tile(c); }

// Start of the workspace: staging of host-side length arrays.
size_t stage_bytes_for(int32_t max_blocks) { return ba_align_up((size_t)(2 * (size_t)max_blocks + 64) * 4, 256); }

struct TableLayout {
  size_t off[24];
  size_t bytes;
};

// Carves the caller's table buffer.  Every array starts on a 16-byte boundary.
TableLayout table_layout(int32_t batch, int32_t B, int32_t T) {
  TableLayout L;
  size_t cur = 0;
  int i = 0;
  auto take = [&](size_t n_bytes) { L.off[i++] = cur; cur = ba_align_up(cur + n_bytes, 16); };
  for (int k = 0; k < 4; ++k) take((size_t)(batch + 1) * 4);  // cu_seq, cu_cache_seq, cu_final_seq, cu_seq_block
  take((size_t)(B + 1) * 4);                                  // cu_block
  for (int k = 0; k < 4; ++k) take((size_t)B * 4);            // block_delta, block_seq, block_kv_begin, block_part_off
  take((size_t)B);                                            // block_is_final
  take((size_t)B * 4);                                        // cache_block
  take((size_t)(B + 1) * 4);                                  // cache_cu
  take((size_t)B * 4);                                        // cache_delta
  for (int k = 0; k < 3; ++k) take((size_t)T * 4);            // tok_block, tok_pos, tok_pos_local
  take((size_t)(B + 1) * 4);                                  // cu_qtile
  take((size_t)(batch + 1) * 4);                              // cu_ftile
  take((size_t)(B + 1) * 4);                                  // cache_tile_cu
  take((size_t)(B + 1) * 4);                                  // cu_ktile
  take(8 * 4);                                                // totals
  take((size_t)B * 64 * 8);                                   // cache_rope: at most 64 rotary pairs per block
  L.bytes = cur;
  return L;
}

}  // namespace

extern "C" {

const char *ba_status_string(ba_status s) {
  switch (s) {
    case BA_OK: return "ok";
    case BA_ERR_INVALID_ARG: return "invalid argument";
    case BA_ERR_SHAPE: return "shape mismatch";
    case BA_ERR_UNSUPPORTED: return "unsupported configuration";
    case BA_ERR_WORKSPACE: return "workspace too small";
    case BA_ERR_CUDA: return "CUDA error";
    case BA_ERR_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown status";
}

ba_status ba_workspace_bytes(const ba_config *cfg, int32_t max_blocks, int32_t max_q_rows, size_t *bytes) {
  ba_status st = check_config(cfg);
  if (st != BA_OK) return st;
  if (!bytes || max_blocks < 1 || max_q_rows < 0) return BA_ERR_INVALID_ARG;
  size_t table = ba_align_up((size_t)max_blocks * cfg->head_dim * 4, 256);
  // split-KV partial results are only used for short query sides (few work items)
  size_t split_rows = (size_t)(max_q_rows < 4096 ? max_q_rows : 4096);
  size_t splits = split_rows * cfg->n_q_heads * (cfg->head_dim + 1) * sizeof(float) * 6;
  size_t stage = stage_bytes_for(max_blocks);
  if (stage < 64 * 1024) stage = 64 * 1024;
  // the backward pass keeps dO . O (fp32 per row and query head) there
  size_t bwd = (size_t)max_q_rows * cfg->n_q_heads * sizeof(float);
  size_t scratch = table > splits ? table : splits;
  if (bwd > scratch) scratch = bwd;
  *bytes = stage + ba_align_up(scratch, 256) + 256;
  return BA_OK;
}

ba_status ba_create(ba_ctx **out, const ba_config *cfg, int device, size_t workspace_bytes) {
  if (!out) return BA_ERR_INVALID_ARG;
  *out = nullptr;
  ba_status st = check_config(cfg);
  if (st != BA_OK) return st;
  int n_dev = 0;
  if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device < 0 || device >= n_dev) {
    cudaGetLastError();
    return BA_ERR_CUDA;
  }
  cudaDeviceProp prop;
  BA_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return BA_ERR_CUDA;  // kernels are built for sm_100a only
  BA_CUDA_TRY(cudaSetDevice(device));
  ba_ctx *ctx = new (std::nothrow) ba_ctx();
  if (!ctx) return BA_ERR_CUDA;
  ctx->cfg = *cfg;
  ctx->device = device;
  ctx->sm_count = prop.multiProcessorCount;
  ctx->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / sqrtf((float)cfg->head_dim);
  ctx->workspace_bytes = workspace_bytes;
  ctx->launches = 0;
  ctx->has_pending = 0;
  ctx->pending_table_bytes = 0;
  ctx->pending_stream = nullptr;
  ctx->seg_delta = nullptr; ctx->seg_rope = nullptr; ctx->seg_rope_blocks = 0;
  ctx->seg_gen = nullptr; ctx->seg_gen_value = 0; ctx->seg_counter = 0;
  ctx->maps = nullptr;
  ctx->side_stream = nullptr; ctx->ev_fork = nullptr; ctx->ev_join = nullptr;
  ctx->workspace = nullptr;
  ctx->dev_status = nullptr;
  if (cudaMalloc(&ctx->dev_status, 256) != cudaSuccess ||
      cudaMemset(ctx->dev_status, 0, 256) != cudaSuccess ||
      (workspace_bytes && cudaMalloc(&ctx->workspace, workspace_bytes) != cudaSuccess) ||
      // launch counters of the attention kernels (below the scratch area): zero once, every launch leaves them zero
      (workspace_bytes >= ba_scratch_offset(ctx) &&
       cudaMemset((char *)ctx->workspace + ba_scratch_offset(ctx) - 256, 0, 256) != cudaSuccess) ||
      cudaStreamCreateWithFlags(&ctx->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming) != cudaSuccess ||
      ba_attend_sm100_setup(ctx) != BA_OK || ba_bwd_sm100_setup(ctx) != BA_OK) {
    cudaGetLastError();
    ba_attend_sm100_teardown(ctx);
    if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
    if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
    if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
    if (ctx->workspace) cudaFree(ctx->workspace);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    delete ctx;
    return BA_ERR_CUDA;
  }
  *out = ctx;
  return BA_OK;
}

ba_status ba_destroy(ba_ctx *ctx) {
  if (!ctx) return BA_ERR_INVALID_ARG;
  cudaSetDevice(ctx->device);
  if (ctx->has_pending) ba_flush_pending(ctx, ctx->pending_stream);   // a queued job is not dropped
  cudaDeviceSynchronize();
  if (ctx->ev_join) cudaEventDestroy(ctx->ev_join);
  if (ctx->ev_fork) cudaEventDestroy(ctx->ev_fork);
  if (ctx->side_stream) cudaStreamDestroy(ctx->side_stream);
  if (ctx->workspace) cudaFree(ctx->workspace);
  if (ctx->dev_status) cudaFree(ctx->dev_status);
  ba_attend_sm100_teardown(ctx);
  delete ctx;
  return BA_OK;
}

ba_status ba_last_device_status(ba_ctx *ctx) {
  if (!ctx) return BA_ERR_INVALID_ARG;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  BA_CUDA_TRY(cudaDeviceSynchronize());
  int32_t h = 0;
  BA_CUDA_TRY(cudaMemcpy(&h, ctx->dev_status, 4, cudaMemcpyDeviceToHost));
  if (h != 0) {
    BA_CUDA_TRY(cudaMemset(ctx->dev_status, 0, 4));
    // a launch that gave up may have left its work counters half-way: back to zero for the next one
    if (ctx->workspace && ctx->workspace_bytes >= ba_scratch_offset(ctx))
      BA_CUDA_TRY(cudaMemset((char *)ctx->workspace + ba_scratch_offset(ctx) - 256, 0, 256));
  }
  return (ba_status)h;
}

int64_t ba_launch_count(const ba_ctx *ctx) { return ctx ? ctx->launches : 0; }

ba_status ba_last_attend_shape(const ba_ctx *ctx, int32_t out[4]) {
  if (!ctx || !out) return BA_ERR_INVALID_ARG;
  for (int i = 0; i < 4; ++i) out[i] = ctx->last_attend[i];
  return BA_OK;
}

ba_status ba_plan_final_attend(int32_t n_sms, int32_t n_pairs, int32_t n_head_chunks, int32_t avg_key_tiles,
                               const int32_t key_tiles[3], int32_t max_partials, int32_t out[3]) {
  if (!key_tiles || !out || n_sms < 1 || n_pairs < 1 || n_head_chunks < 1 || avg_key_tiles < 1) return BA_ERR_INVALID_ARG;
  const ba_split_plan plan = ba_plan_splits(n_sms, (long long)n_pairs * n_head_chunks, n_pairs, n_head_chunks,
                                            avg_key_tiles, key_tiles, max_partials);
  out[0] = plan.n_splits; out[1] = plan.balanced; out[2] = plan.bal_len;
  return BA_OK;
}

ba_status ba_segments_bytes(int32_t batch, int32_t n_blocks, int32_t n_tokens, size_t *bytes) {
  if (!bytes || batch < 1 || n_blocks < batch || n_tokens < n_blocks) return BA_ERR_INVALID_ARG;
  *bytes = table_layout(batch, n_blocks, n_tokens).bytes;
  return BA_OK;
}

ba_status ba_segment(ba_ctx *ctx, const int32_t *block_lens, const int32_t *seq_nblocks,
                     int32_t batch, int32_t n_blocks, int32_t n_tokens, ba_mode mode,
                     void *table_buf, size_t table_bytes, ba_segments *out, void *stream) {
  if (!ctx || !block_lens || !seq_nblocks || !table_buf || !out) return BA_ERR_INVALID_ARG;
  if (mode != BA_MODE_BLOCK && mode != BA_MODE_FULL) return BA_ERR_INVALID_ARG;
  if (batch < 1 || n_blocks < batch || n_tokens < n_blocks) return BA_ERR_INVALID_ARG;
  if (!aligned16(table_buf)) return BA_ERR_INVALID_ARG;
  TableLayout L = table_layout(batch, n_blocks, n_tokens);
  if (table_bytes < L.bytes) return BA_ERR_SHAPE;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  cudaStream_t s = (cudaStream_t)stream;

  const int32_t *d_lens = block_lens, *d_nb = seq_nblocks;
  const bool host_lens = is_host_pointer(block_lens), host_nb = is_host_pointer(seq_nblocks);
  if (host_lens != host_nb) return BA_ERR_INVALID_ARG;
  if (host_lens) {
    long long sum = 0, nb_sum = 0;
    for (int b = 0; b < n_blocks; ++b) { if (block_lens[b] < 1) return BA_ERR_INVALID_ARG; sum += block_lens[b]; }
    for (int q = 0; q < batch; ++q) { if (seq_nblocks[q] < 1) return BA_ERR_INVALID_ARG; nb_sum += seq_nblocks[q]; }
    if (sum != n_tokens || nb_sum != n_blocks) return BA_ERR_INVALID_ARG;
    size_t need = (size_t)(n_blocks + batch) * 4;
    // staging area: the start of the workspace, up to the launch counters below the scratch area
    if (!ctx->workspace || need > ctx->workspace_bytes ||
        (ctx->workspace_bytes >= ba_scratch_offset(ctx) && need > ba_scratch_offset(ctx) - 256))
      return BA_ERR_WORKSPACE;
    int32_t *stage = (int32_t *)ctx->workspace;
    BA_CUDA_TRY(cudaMemcpyAsync(stage, block_lens, (size_t)n_blocks * 4, cudaMemcpyHostToDevice, s));
    BA_CUDA_TRY(cudaMemcpyAsync(stage + n_blocks, seq_nblocks, (size_t)batch * 4, cudaMemcpyHostToDevice, s));
    d_lens = stage;
    d_nb = stage + n_blocks;
  }

  char *base = (char *)table_buf;
  int i = 0;
  memset(out, 0, sizeof(*out));
  out->batch = batch; out->n_blocks = n_blocks; out->n_tokens = n_tokens;
  out->n_cached_blocks = n_blocks - batch;
  out->mode = mode;
  out->q_tile_tokens = q_tile_tokens(ctx->cfg);
  if (host_lens) {   // lengths known here: the attention launches can be sized exactly
    const int tt = out->q_tile_tokens;
    long long items = 0, fitems = 0;
    for (int b = 0; b < n_blocks; ++b) items += (block_lens[b] + tt - 1) / tt;
    for (int q = 0, b = 0; q < batch; ++q) { b += seq_nblocks[q]; fitems += (block_lens[b - 1] + tt - 1) / tt; }
    out->n_prompt_items = (int32_t)items; out->n_final_items = (int32_t)fitems;
    // key tiles per item of the final blocks (the counting of the attention kernel, done here on the host)
    long long sum[2] = {0, 0}, mn[2] = {INT32_MAX, INT32_MAX}, mx[2] = {0, 0};
    for (int q = 0, b = 0; q < batch; ++q) {
      long long cached = 0, walked = 0;
      for (int c = 0; c + 1 < seq_nblocks[q]; ++c) { cached += block_lens[b + c]; walked += (block_lens[b + c] + 127) / 128; }
      b += seq_nblocks[q];
      const long long ct[2] = {(cached + 127) / 128, walked};
      const int fin = block_lens[b - 1];
      for (int r0 = 0; r0 < fin; r0 += tt) {
        const long long own = (std::min(fin, r0 + tt) + 127) / 128;
        for (int k = 0; k < 2; ++k) {
          const long long n = ct[k] + own;
          sum[k] += n; mn[k] = std::min(mn[k], n); mx[k] = std::max(mx[k], n);
        }
      }
    }
    for (int k = 0; k < 2; ++k) {
      const bool fits = sum[k] <= INT32_MAX;
      out->final_key_tiles[3 * k] = fits ? (int32_t)sum[k] : 0;
      out->final_key_tiles[3 * k + 1] = fits ? (int32_t)mn[k] : 0;
      out->final_key_tiles[3 * k + 2] = fits ? (int32_t)mx[k] : 0;
    }
  }
  auto next = [&]() { return (int32_t *)(base + L.off[i++]); };
  out->cu_seq = next(); out->cu_cache_seq = next(); out->cu_final_seq = next(); out->cu_seq_block = next();
  out->cu_block = next();
  out->block_delta = next(); out->block_seq = next(); out->block_kv_begin = next(); out->block_part_off = next();
  out->block_is_final = (uint8_t *)next();
  out->cache_block = next(); out->cache_cu = next(); out->cache_delta = next();
  out->tok_block = next(); out->tok_pos = next(); out->tok_pos_local = next();
  out->cu_qtile = next(); out->cu_ftile = next(); out->cache_tile_cu = next(); out->cu_ktile = next();
  out->totals = next();
  out->cache_rope = (float *)next();
  ctx->seg_delta = nullptr; ctx->seg_rope = nullptr; ctx->seg_rope_blocks = 0; ctx->seg_gen = nullptr;
  // Every call stamps its tables (totals[6]) with a value that differs from call to call and from
  // context to context: a later re-encoding that wants to reuse the rotation table stored with the
  // tables can tell on the device whether the buffer still holds this call's tables.
  ctx->seg_counter += 1;
  const int32_t gen = (int32_t)((((uint32_t)((uintptr_t)ctx >> 6)) * 0x9E3779B1u +
                                 (uint32_t)ctx->seg_counter * 0x85EBCA6Bu) | 1u);
  ba_status st = ba_segment_launch(ctx, d_lens, d_nb, batch, n_blocks, n_tokens, mode, gen, out, s);
  if (st != BA_OK || out->n_cached_blocks == 0) return st;
  // rotations of the cached blocks (the same angle table ba_reencode_k builds), once per prompt
  st = ba_reencode_table_launch(ctx, out->cache_delta, out->n_cached_blocks, (float2 *)out->cache_rope, s);
  if (st == BA_OK) {
    ctx->seg_delta = out->cache_delta; ctx->seg_rope = (const float2 *)out->cache_rope;
    ctx->seg_rope_blocks = out->n_cached_blocks;
    ctx->seg_gen = out->totals + 6; ctx->seg_gen_value = gen;
  }
  return st;
}

static ba_status check_reencode_args(ba_ctx *ctx, const void *k_src, const int32_t *src_off, int32_t n_src_rows,
                                     void *k_dst, const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                                     int32_t n_rows, bool *nothing_to_do) {
  *nothing_to_do = false;
  if (!ctx) return BA_ERR_INVALID_ARG;
  if (n_blocks < 0 || n_rows < 0 || n_src_rows < 0) return BA_ERR_INVALID_ARG;
  if (n_blocks == 0 || n_rows == 0) { *nothing_to_do = true; return BA_OK; }   // nothing cached
  if (!k_src || !k_dst || !cu || !delta) return BA_ERR_INVALID_ARG;
  if (!aligned16(k_src) || !aligned16(k_dst)) return BA_ERR_INVALID_ARG;
  if (k_src == k_dst && src_off) return BA_ERR_INVALID_ARG;  // a gather cannot run in place
  return BA_OK;
}

// The angle table of a call sits at the end of the workspace, below the table of a queued job.
static ba_status place_table(ba_ctx *ctx, int32_t n_blocks, float2 **table, size_t *bytes) {
  const size_t need = ba_align_up((size_t)n_blocks * ctx->cfg.head_dim * 4, 256);  // n_blocks * d/2 * sizeof(float2)
  if (!ctx->workspace || ba_scratch_offset(ctx) + need + ctx->pending_table_bytes > ctx->workspace_bytes)
    return BA_ERR_WORKSPACE;
  *table = (float2 *)((char *)ctx->workspace + (ctx->workspace_bytes - ctx->pending_table_bytes - need) / 256 * 256);
  *bytes = need;
  return BA_OK;
}

ba_status ba_reencode_k(ba_ctx *ctx, const void *k_src, const int32_t *src_off, int32_t n_src_rows,
                        void *k_dst, const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                        int32_t n_rows, void *stream) {
  bool nothing;
  ba_status st = check_reencode_args(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, &nothing);
  if (st != BA_OK || nothing) return st;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  if (delta == ctx->seg_delta && n_blocks == ctx->seg_rope_blocks) {   // the table ba_segment built is for these deltas
    ba_reencode_job job =
        ba_make_reencode_job(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, ctx->seg_rope);
    job.gen = ctx->seg_gen; job.gen_expected = ctx->seg_gen_value;
    return ba_reencode_main_launch(ctx, job, (cudaStream_t)stream);
  }
  float2 *table; size_t bytes;
  st = place_table(ctx, n_blocks, &table, &bytes);
  if (st != BA_OK) return st;
  return ba_reencode_launch(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, table,
                            (cudaStream_t)stream);
}

ba_status ba_reencode_k_deferred(ba_ctx *ctx, const void *k_src, const int32_t *src_off, int32_t n_src_rows,
                                 void *k_dst, const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                                 int32_t n_rows, void *stream) {
  bool nothing;
  ba_status st = check_reencode_args(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, &nothing);
  if (st != BA_OK || nothing) return st;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  st = ba_flush_pending(ctx, (cudaStream_t)stream);          // one job may be queued at a time
  if (st != BA_OK) return st;
  const float2 *table_used;
  size_t bytes = 0;
  if (delta == ctx->seg_delta && n_blocks == ctx->seg_rope_blocks) {
    table_used = ctx->seg_rope;
  } else {
    float2 *table;
    st = place_table(ctx, n_blocks, &table, &bytes);
    if (st != BA_OK) return st;
    st = ba_reencode_table_launch(ctx, delta, n_blocks, table, (cudaStream_t)stream);
    if (st != BA_OK) return st;
    table_used = table;
  }
  ctx->pending = ba_make_reencode_job(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, table_used);
  if (table_used == ctx->seg_rope) { ctx->pending.gen = ctx->seg_gen; ctx->pending.gen_expected = ctx->seg_gen_value; }
  ctx->has_pending = 1;
  ctx->pending_table_bytes = bytes;
  ctx->pending_stream = (cudaStream_t)stream;
  return BA_OK;
}

ba_status ba_flush(ba_ctx *ctx, void *stream) {
  if (!ctx) return BA_ERR_INVALID_ARG;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  return ba_flush_pending(ctx, (cudaStream_t)stream);
}

static ba_status check_attend_common(ba_ctx *ctx, const void *q, const void *k, const void *v, void *o,
                                     const ba_segments *seg, ba_mode mode, ba_out_dtype od) {
  if (!ctx || !q || !k || !v || !o || !seg) return BA_ERR_INVALID_ARG;
  if (mode != BA_MODE_BLOCK && mode != BA_MODE_FULL) return BA_ERR_INVALID_ARG;
  if ((int)mode != seg->mode) return BA_ERR_INVALID_ARG;
  if (od != BA_OUT_BF16 && od != BA_OUT_F32) return BA_ERR_INVALID_ARG;
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(o)) return BA_ERR_INVALID_ARG;
  if (!seg->totals || !seg->cu_block || !seg->tok_block) return BA_ERR_INVALID_ARG;
  return BA_OK;
}

ba_status ba_block_prefill(ba_ctx *ctx, const void *q, const void *k, const void *v, void *o,
                           float *lse, const ba_segments *seg, ba_mode mode,
                           ba_out_dtype out_dtype, void *stream) {
  ba_status st = check_attend_common(ctx, q, k, v, o, seg, mode, out_dtype);
  if (st != BA_OK) return st;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  ba_attend_args a;
  memset(&a, 0, sizeof(a));
  a.q = (const __nv_bfloat16 *)q; a.k = (const __nv_bfloat16 *)k; a.v = (const __nv_bfloat16 *)v;
  a.o = o; a.lse = lse; a.n_q_rows = seg->n_tokens; a.n_kv_rows = seg->n_tokens;
  a.out_f32 = out_dtype == BA_OUT_F32;
  a.final_only = 0;
  return ba_attend_launch(ctx, a, seg, (cudaStream_t)stream);
}

ba_status ba_final_attend(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                          int32_t n_final_rows, const void *k_cache, const void *v_cache,
                          int32_t n_cache_rows, const int32_t *v_src_off, int32_t n_v_rows,
                          void *o, float *lse, const ba_segments *seg, ba_mode mode,
                          ba_out_dtype out_dtype, void *stream) {
  ba_status st = check_attend_common(ctx, q_f, k_f, v_f, o, seg, mode, out_dtype);
  if (st != BA_OK) return st;
  if (n_final_rows < 0 || n_cache_rows < 0) return BA_ERR_INVALID_ARG;
  if (n_cache_rows > 0 && (!k_cache || !v_cache || !aligned16(k_cache) || !aligned16(v_cache)))
    return BA_ERR_INVALID_ARG;
  if (v_src_off && n_v_rows < 1) return BA_ERR_INVALID_ARG;
  // the tables describe n_tokens rows: the caller's final and cached tensors must add up to them
  if ((long long)n_final_rows + n_cache_rows != seg->n_tokens) return BA_ERR_SHAPE;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  ba_attend_args a;
  memset(&a, 0, sizeof(a));
  a.q = (const __nv_bfloat16 *)q_f; a.k = (const __nv_bfloat16 *)k_f; a.v = (const __nv_bfloat16 *)v_f;
  a.o = o; a.lse = lse; a.n_q_rows = n_final_rows; a.n_kv_rows = n_final_rows;
  a.k_cache = (const __nv_bfloat16 *)k_cache; a.v_cache = (const __nv_bfloat16 *)v_cache;
  a.n_cache_rows = n_cache_rows; a.n_v_rows = v_src_off ? n_v_rows : n_cache_rows;
  a.v_src_off = v_src_off;
  a.out_f32 = out_dtype == BA_OUT_F32;
  a.final_only = 1;
  return ba_attend_launch(ctx, a, seg, (cudaStream_t)stream);
}

ba_status ba_final_attend_fused(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                                int32_t n_final_rows, const void *k_src, const void *v_src,
                                int32_t n_src_rows, const int32_t *src_off, int32_t n_cache_rows,
                                void *k_out, void *o, float *lse, const ba_segments *seg, ba_mode mode,
                                ba_out_dtype out_dtype, void *stream) {
  ba_status st = check_attend_common(ctx, q_f, k_f, v_f, o, seg, mode, out_dtype);
  if (st != BA_OK) return st;
  if (n_final_rows < 0 || n_cache_rows < 0 || n_src_rows < 0) return BA_ERR_INVALID_ARG;
  if (n_cache_rows > 0) {
    if (!k_src || !v_src || !aligned16(k_src) || !aligned16(v_src)) return BA_ERR_INVALID_ARG;
    if (n_src_rows < 1 || !seg->cache_rope || !seg->cache_tile_cu) return BA_ERR_INVALID_ARG;
    if (!src_off && n_src_rows < n_cache_rows) return BA_ERR_INVALID_ARG;
    if (k_out && (!aligned16(k_out) || k_out == k_src)) return BA_ERR_INVALID_ARG;   // the attention reads k_src meanwhile
  }
  if ((long long)n_final_rows + n_cache_rows != seg->n_tokens) return BA_ERR_SHAPE;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  ba_attend_args a;
  memset(&a, 0, sizeof(a));
  a.q = (const __nv_bfloat16 *)q_f; a.k = (const __nv_bfloat16 *)k_f; a.v = (const __nv_bfloat16 *)v_f;
  a.o = o; a.lse = lse; a.n_q_rows = n_final_rows; a.n_kv_rows = n_final_rows;
  a.k_cache = (const __nv_bfloat16 *)k_src; a.v_cache = (const __nv_bfloat16 *)v_src;
  a.n_cache_rows = n_cache_rows;
  a.fused = 1;
  a.k_src_off = src_off; a.n_k_rows = n_src_rows;
  a.k_out = n_cache_rows > 0 ? k_out : nullptr;
  // values: addressed like the keys.  The kernel's value map covers n_v_rows rows when an offset table is given.
  a.v_src_off = src_off; a.n_v_rows = n_src_rows;
  a.out_f32 = out_dtype == BA_OUT_F32;
  a.final_only = 1;
  return ba_attend_launch(ctx, a, seg, (cudaStream_t)stream);
}


ba_status ba_block_prefill_bwd(ba_ctx *ctx, const void *q, const void *k, const void *v, const void *o,
                               const float *lse, const void *d_o, void *dq, void *dk, void *dv,
                               const ba_segments *seg, ba_mode mode, ba_out_dtype grad_dtype, void *stream) {
  ba_status st = check_attend_common(ctx, q, k, v, dq, seg, mode, grad_dtype);
  if (st != BA_OK) return st;
  if (!o || !lse || !d_o || !dk || !dv) return BA_ERR_INVALID_ARG;
  if (!aligned16(o) || !aligned16(d_o) || !aligned16(dk) || !aligned16(dv)) return BA_ERR_INVALID_ARG;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  st = ba_flush_pending(ctx, (cudaStream_t)stream);      // a queued re-encoding job does not ride along here
  if (st != BA_OK) return st;
  return ba_bwd_sm100_launch(ctx, q, k, v, o, lse, d_o, dq, dk, dv, grad_dtype == BA_OUT_F32, seg, (int)mode,
                             (cudaStream_t)stream);
}

static ba_status check_pages(const ba_page_table *pg) {
  if (!pg || !pg->page_cu || !pg->page_idx) return BA_ERR_INVALID_ARG;
  if (pg->page_rows < 16 || pg->page_rows > 65536 || (pg->page_rows & (pg->page_rows - 1))) return BA_ERR_UNSUPPORTED;
  if (pg->n_pages < 1 || (long long)pg->n_pages * pg->page_rows > 0x7fffffffLL) return BA_ERR_INVALID_ARG;
  return BA_OK;
}

ba_status ba_reencode_k_paged(ba_ctx *ctx, const void *k_pool, const ba_page_table *pages, void *k_dst,
                              const int32_t *cu, const int32_t *delta, int32_t n_blocks, int32_t n_rows,
                              void *stream) {
  ba_status st = check_pages(pages);
  if (st != BA_OK) return st;
  const int32_t n_src_rows = pages->n_pages * pages->page_rows;
  bool nothing;
  st = check_reencode_args(ctx, k_pool, nullptr, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, &nothing);
  if (st != BA_OK || nothing) return st;
  if (k_pool == k_dst) return BA_ERR_INVALID_ARG;            // a gather cannot run in place
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  const bool reuse = delta == ctx->seg_delta && n_blocks == ctx->seg_rope_blocks;
  float2 *table = nullptr; size_t bytes;
  if (!reuse) {
    st = place_table(ctx, n_blocks, &table, &bytes);
    if (st != BA_OK) return st;
    st = ba_reencode_table_launch(ctx, delta, n_blocks, table, (cudaStream_t)stream);
    if (st != BA_OK) return st;
  }
  ba_reencode_job job = ba_make_reencode_job(ctx, k_pool, nullptr, n_src_rows, k_dst, cu, delta, n_blocks, n_rows,
                                             reuse ? ctx->seg_rope : table);
  if (reuse) { job.gen = ctx->seg_gen; job.gen_expected = ctx->seg_gen_value; }
  job.page_cu = pages->page_cu; job.page_idx = pages->page_idx;
  job.page_lg = 0;
  while ((1 << job.page_lg) < pages->page_rows) ++job.page_lg;
  return ba_reencode_main_launch(ctx, job, (cudaStream_t)stream);
}

ba_status ba_final_attend_paged(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                                int32_t n_final_rows, const void *k_cache, int32_t n_cache_rows,
                                const void *v_pool, const ba_page_table *pages, void *o, float *lse,
                                const ba_segments *seg, ba_mode mode, ba_out_dtype out_dtype, void *stream) {
  ba_status st = check_attend_common(ctx, q_f, k_f, v_f, o, seg, mode, out_dtype);
  if (st != BA_OK) return st;
  if (n_final_rows < 0 || n_cache_rows < 0) return BA_ERR_INVALID_ARG;
  if ((long long)n_final_rows + n_cache_rows != seg->n_tokens) return BA_ERR_SHAPE;
  ba_attend_args a;
  memset(&a, 0, sizeof(a));
  if (n_cache_rows > 0) {
    st = check_pages(pages);
    if (st != BA_OK) return st;
    if (!k_cache || !v_pool || !aligned16(k_cache) || !aligned16(v_pool) || !seg->cache_tile_cu) return BA_ERR_INVALID_ARG;
    a.page_rows = pages->page_rows; a.page_cu = pages->page_cu; a.page_idx = pages->page_idx;
    a.n_v_rows = pages->n_pages * pages->page_rows;
  }
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  a.q = (const __nv_bfloat16 *)q_f; a.k = (const __nv_bfloat16 *)k_f; a.v = (const __nv_bfloat16 *)v_f;
  a.o = o; a.lse = lse; a.n_q_rows = n_final_rows; a.n_kv_rows = n_final_rows;
  a.k_cache = (const __nv_bfloat16 *)k_cache; a.v_cache = (const __nv_bfloat16 *)v_pool;
  a.n_cache_rows = n_cache_rows;
  a.out_f32 = out_dtype == BA_OUT_F32;
  a.final_only = 1;
  return ba_attend_launch(ctx, a, seg, (cudaStream_t)stream);
}

ba_status ba_final_attend_fused_paged(ba_ctx *ctx, const void *q_f, const void *k_f, const void *v_f,
                                      int32_t n_final_rows, const void *k_pool, const void *v_pool,
                                      const ba_page_table *pages, int32_t n_cache_rows, void *k_out,
                                      void *o, float *lse, const ba_segments *seg, ba_mode mode,
                                      ba_out_dtype out_dtype, void *stream) {
  ba_status st = check_attend_common(ctx, q_f, k_f, v_f, o, seg, mode, out_dtype);
  if (st != BA_OK) return st;
  if (n_final_rows < 0 || n_cache_rows < 0) return BA_ERR_INVALID_ARG;
  if ((long long)n_final_rows + n_cache_rows != seg->n_tokens) return BA_ERR_SHAPE;
  ba_attend_args a;
  memset(&a, 0, sizeof(a));
  if (n_cache_rows > 0) {
    st = check_pages(pages);
    if (st != BA_OK) return st;
    if (!k_pool || !v_pool || !aligned16(k_pool) || !aligned16(v_pool)) return BA_ERR_INVALID_ARG;
    if (!seg->cache_rope || !seg->cache_tile_cu) return BA_ERR_INVALID_ARG;
    if (k_out && (!aligned16(k_out) || k_out == k_pool)) return BA_ERR_INVALID_ARG;
    a.page_rows = pages->page_rows; a.page_cu = pages->page_cu; a.page_idx = pages->page_idx;
    a.n_k_rows = a.n_v_rows = pages->n_pages * pages->page_rows;
    a.k_out = k_out;
  }
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  a.q = (const __nv_bfloat16 *)q_f; a.k = (const __nv_bfloat16 *)k_f; a.v = (const __nv_bfloat16 *)v_f;
  a.o = o; a.lse = lse; a.n_q_rows = n_final_rows; a.n_kv_rows = n_final_rows;
  a.k_cache = (const __nv_bfloat16 *)k_pool; a.v_cache = (const __nv_bfloat16 *)v_pool;
  a.n_cache_rows = n_cache_rows;
  a.fused = 1;
  a.out_f32 = out_dtype == BA_OUT_F32;
  a.final_only = 1;
  return ba_attend_launch(ctx, a, seg, (cudaStream_t)stream);
}

}  // extern "C"

ba_status ba_attend_launch(ba_ctx *ctx, const ba_attend_args &a, const ba_segments *seg,
                           cudaStream_t stream) {
  if (a.n_q_rows == 0) return ba_flush_pending(ctx, stream);   // no attention launch to ride along with
  return ba_attend_sm100_launch(ctx, a, seg, stream);
}

// Position re-encoding of cached keys (Section 2.3, Eq. 1-3).
//
// The paper resets a cached key to position zero (Eq. 2) and then rotates it to
// its new position (Eq. 3); both are rotations of the same 2x2 blocks, so their
// product is one rotation by the position difference.  Every token of a block
// moves by the same difference (the block's new start, because cached blocks
// start at zero), hence one (cos, sin) pair per (block, rotary pair) serves the
// whole block.
//
// Kernel 1 builds that table in fp64 (angles reach tens of thousands of radians,
// far beyond what fast fp32 sin/cos can reduce) and stores it as fp32.
// Kernel 2 is a pure bandwidth kernel: every thread moves 16-byte vectors
// (8 bf16) and keeps its column while it walks down a few rows, rotating in fp32 and rounding
// once to bf16; small CTAs (one row of vectors wide) measured fastest.
#include "ba_common.cuh"
#include "ba_reencode_dev.cuh"

namespace {

__global__ void __launch_bounds__(128)
ba_rope_table_kernel(const int32_t *__restrict__ delta, int n_blocks, int half_dim,
                     double neg2_over_d_log2_base, float2 *__restrict__ table) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_blocks * half_dim) return;
  int c = i / half_dim, m = i - c * half_dim;
  // theta_m = base^(-2m/d) = 2^(m * (-2/d) * log2(base))
  double theta = exp2((double)m * neg2_over_d_log2_base);
  double a = (double)delta[c] * theta;
  double s, co;
  sincos(a, &s, &co);
  table[i] = make_float2((float)co, (float)s);
}

// A CTA takes kPasses consecutive groups of rows; its threads keep their column and walk down the
// rows, kRows loads in flight each, so the per-thread set-up (column arithmetic, block search, table
// fetch) is paid once per kPasses * kRows rows.
template <int kLayout, int kRows, int kPasses>
__global__ void __launch_bounds__(512)
ba_reencode_kernel(const ba_reencode_job job, int units_shift, int32_t *status) {
  // units per row is a power of two for every head count that is one (units_shift >= 0): shifts, no divisions
  const int units_per_row = (kLayout == BA_ROPE_ADJACENT) ? job.row_vecs : (job.row_vecs >> 1);
  const int row_step = units_shift >= 0 ? (int)(blockDim.x >> units_shift) : (int)(blockDim.x / units_per_row);
  const int u = units_shift >= 0 ? (int)(threadIdx.x & (units_per_row - 1)) : (int)(threadIdx.x % units_per_row);
  const int rsub = units_shift >= 0 ? (int)(threadIdx.x >> units_shift) : (int)(threadIdx.x / units_per_row);
  const int total_rows = min(job.n_rows, __ldg(job.cu + job.n_blocks));
  const int cta_row0 = blockIdx.x * (row_step * kRows * kPasses);
  if (job.gen && __ldg(job.gen) != job.gen_expected) {     // the rotation table is not the one this job was given
    if (threadIdx.x == 0) ba_record_status(status, BA_ERR_INVALID_ARG);
    return;
  }
  // the block of the CTA's first row is searched once and shared; the threads walk forward from it
  __shared__ int s_c;
  if (threadIdx.x == 0) {
    int c = upper_bound_i32(job.cu, job.n_blocks + 1, min(cta_row0, max(total_rows - 1, 0))) - 1;
    s_c = min(max(c, 0), job.n_blocks - 1);
  }
  __syncthreads();
  int row0 = cta_row0 + rsub;
  if (row0 >= total_rows) return;
  ba_reencode_state st;
  ba_reencode_state_init<kLayout>(job, u, st);
  st.c = s_c;
  st.c_begin = __ldg(job.cu + st.c);
  st.c_end = __ldg(job.cu + st.c + 1);
  st.shift = job.src_off ? (long long)__ldg(job.src_off + st.c) - st.c_begin : 0;
  st.page0 = job.page_cu ? __ldg(job.page_cu + st.c) : 0;
#pragma unroll 1
  for (int pass = 0; pass < kPasses && row0 < total_rows; ++pass, row0 += row_step * kRows)
    ba_reencode_rows<kLayout, kRows>(job, st, row0, row_step, total_rows, status);
}

}  // namespace

ba_status ba_reencode_table_launch(ba_ctx *ctx, const int32_t *delta, int32_t n_blocks, float2 *table,
                                   cudaStream_t stream) {
  const int D = ctx->cfg.head_dim, half = D / 2;
  const double k = -2.0 / (double)D * log2(ctx->cfg.rope_theta);
  const int n = n_blocks * half;
  ba_rope_table_kernel<<<(n + 127) / 128, 128, 0, stream>>>(delta, n_blocks, half, k, table);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 1;
  return BA_OK;
}

ba_reencode_job ba_make_reencode_job(const ba_ctx *ctx, const void *k_src, const int32_t *src_off,
                                     int32_t n_src_rows, void *k_dst, const int32_t *cu, const int32_t *delta,
                                     int32_t n_blocks, int32_t n_rows, const float2 *table) {
  ba_reencode_job job;
  job.src = (const uint4 *)k_src; job.dst = (uint4 *)k_dst; job.src_off = src_off; job.cu = cu; job.delta = delta;
  job.table = table; job.n_src_rows = n_src_rows; job.n_blocks = n_blocks; job.n_rows = n_rows;
  job.head_dim = ctx->cfg.head_dim; job.row_vecs = ctx->cfg.n_kv_heads * ctx->cfg.head_dim / 8;
  job.layout = ctx->cfg.rope_layout;
  job.gen = nullptr; job.gen_expected = 0;
  job.page_cu = nullptr; job.page_idx = nullptr; job.page_lg = 0;
  return job;
}

ba_status ba_reencode_main_launch(ba_ctx *ctx, const ba_reencode_job &job, cudaStream_t stream) {
  constexpr int kRows = 1;                  // rows in flight per thread
  const bool adjacent = job.layout == BA_ROPE_ADJACENT;
  const int units = adjacent ? job.row_vecs : job.row_vecs / 2;
  // threads per CTA: a multiple of the units per row, close to 128
  int threads = units >= 128 ? units : (128 / units) * units;
  int units_shift = -1;                       // log2(units) when it is a power of two
  for (int k = 0; k < 12; ++k) if ((1 << k) == units) units_shift = k;
  if (threads > 512) return BA_ERR_UNSUPPORTED;   // more than 4096 bf16 per row
  constexpr int kPasses = 4;                // consecutive row groups per CTA
  const int rows_per_cta = (threads / units) * kRows * kPasses;
  const int grid = (job.n_rows + rows_per_cta - 1) / rows_per_cta;
  if (adjacent)
    ba_reencode_kernel<BA_ROPE_ADJACENT, kRows, kPasses><<<grid, threads, 0, stream>>>(job, units_shift, ctx->dev_status);
  else
    ba_reencode_kernel<BA_ROPE_HALF, kRows, kPasses><<<grid, threads, 0, stream>>>(job, units_shift, ctx->dev_status);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 1;
  return BA_OK;
}

ba_status ba_reencode_launch(ba_ctx *ctx, const void *k_src, const int32_t *src_off,
                             int32_t n_src_rows, void *k_dst, const int32_t *cu,
                             const int32_t *delta, int32_t n_blocks, int32_t n_rows, float2 *table,
                             cudaStream_t stream) {
  ba_status st = ba_reencode_table_launch(ctx, delta, n_blocks, table, stream);
  if (st != BA_OK) return st;
  return ba_reencode_main_launch(
      ctx, ba_make_reencode_job(ctx, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows, table), stream);
}

ba_status ba_flush_pending(ba_ctx *ctx, cudaStream_t stream) {
  if (!ctx->has_pending) return BA_OK;
  ctx->has_pending = 0;
  ctx->pending_table_bytes = 0;
  return ba_reencode_main_launch(ctx, ctx->pending, stream);
}

// ---------------------------------------------------------------------------
// Allocation-free variant.  The angle table lives in a fixed array that is part
// of the library image; each device that loads the library gets its own copy.
// ---------------------------------------------------------------------------
#include <mutex>

namespace {

constexpr int kNoallocMaxDevices = 64;
// 4096 blocks x 64 rotary pairs x (cos, sin) = 2 MiB per device
static __device__ __align__(256) float2 ba_noalloc_table[BA_NOALLOC_MAX_BLOCKS * 64];
// Receives "bad source row" reports when the caller passes no status word.
static __device__ int32_t ba_noalloc_status_sink;

// In host code the two names above are host-side handles, not device addresses.
// The addresses a kernel can use are looked up once per device and kept here.
float2 *g_noalloc_table[kNoallocMaxDevices];
int32_t *g_noalloc_sink[kNoallocMaxDevices];
std::mutex g_noalloc_mutex;

}  // namespace

extern "C" ba_status ba_reencode_k_noalloc(const ba_config *cfg, int device, const void *k_src,
                                           const int32_t *src_off, int32_t n_src_rows, void *k_dst,
                                           const int32_t *cu, const int32_t *delta, int32_t n_blocks,
                                           int32_t n_rows, int32_t *status_word, void *stream) {
  if (!cfg) return BA_ERR_INVALID_ARG;
  if (cfg->head_dim != 64 && cfg->head_dim != 128) return BA_ERR_UNSUPPORTED;
  if (cfg->n_kv_heads < 1) return BA_ERR_UNSUPPORTED;
  if (cfg->rope_layout != BA_ROPE_ADJACENT && cfg->rope_layout != BA_ROPE_HALF) return BA_ERR_INVALID_ARG;
  if (!(cfg->rope_theta > 1.0)) return BA_ERR_INVALID_ARG;
  if (device < 0 || device >= kNoallocMaxDevices) return BA_ERR_INVALID_ARG;
  {
    int n_dev = 0;
    if (cudaGetDeviceCount(&n_dev) != cudaSuccess || device >= n_dev) { cudaGetLastError(); return BA_ERR_CUDA; }
  }
  if (n_blocks < 0 || n_rows < 0 || n_src_rows < 0) return BA_ERR_INVALID_ARG;
  if (n_blocks > BA_NOALLOC_MAX_BLOCKS) return BA_ERR_WORKSPACE;   // built-in table too small
  if (n_blocks == 0 || n_rows == 0) return BA_OK;
  if (!k_src || !k_dst || !cu || !delta) return BA_ERR_INVALID_ARG;
  if (((uintptr_t)k_src | (uintptr_t)k_dst) & 15u) return BA_ERR_INVALID_ARG;
  if (k_src == k_dst && src_off) return BA_ERR_INVALID_ARG;
  BA_CUDA_TRY(cudaSetDevice(device));
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_table[device]) {   // first call on this device, which is current
      float2 *t = nullptr;
      int32_t *sink = nullptr;
      BA_CUDA_TRY(cudaGetSymbolAddress((void **)&t, ba_noalloc_table));
      BA_CUDA_TRY(cudaGetSymbolAddress((void **)&sink, ba_noalloc_status_sink));
      g_noalloc_sink[device] = sink;
      g_noalloc_table[device] = t;
    }
  }
  // A context on the stack carries the configuration to the shared launch code; nothing is allocated.
  ba_ctx tmp;
  tmp.cfg = *cfg;
  tmp.device = device;
  tmp.sm_count = 0;
  tmp.scale = 0.f;
  tmp.workspace = nullptr;
  tmp.workspace_bytes = 0;
  tmp.dev_status = status_word ? status_word : g_noalloc_sink[device];
  tmp.launches = 0;
  tmp.has_pending = 0;
  tmp.pending_table_bytes = 0;
  tmp.pending_stream = nullptr;
  tmp.seg_delta = nullptr; tmp.seg_rope = nullptr; tmp.seg_rope_blocks = 0;
  tmp.seg_gen = nullptr; tmp.seg_gen_value = 0; tmp.seg_counter = 0; tmp.maps = nullptr;
  tmp.side_stream = nullptr; tmp.ev_fork = nullptr; tmp.ev_join = nullptr;
  return ba_reencode_launch(&tmp, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows,
                            g_noalloc_table[device], (cudaStream_t)stream);
}

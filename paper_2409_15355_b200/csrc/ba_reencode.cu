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
// (8 bf16), several rows in flight, rotating in fp32 and rounding once to bf16.
#include "ba_common.cuh"

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

__device__ __forceinline__ int upper_bound_i32(const int32_t *a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(a + mid) <= x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__device__ __forceinline__ void rot2(float x, float y, float2 cs, float &xo, float &yo) {
  xo = fmaf(x, cs.x, -y * cs.y);
  yo = fmaf(x, cs.y, y * cs.x);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t *>(&v);
}

__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// ADJACENT layout: a 16-byte vector holds rotary pairs 4v..4v+3 of one head.
// HALF layout: the vector at column c (< d/2) pairs with the vector at c + d/2,
// a thread moves both.
// A thread owns one vector column (ADJACENT) or one column pair (HALF) of kRows rows.
template <int kLayout, int kRows>
__global__ void __launch_bounds__(512)
ba_reencode_kernel(const uint4 *src, uint4 *dst,  // may alias (in place): no __restrict__
                   const int32_t *__restrict__ src_off, int n_src_rows,
                   const int32_t *__restrict__ cu, const int32_t *__restrict__ delta, int n_blocks,
                   int n_rows, int head_dim, int row_vecs /* uint4 per row */,
                   const float2 *__restrict__ table, int32_t *status) {
  const int half_dim = head_dim >> 1;
  const int head_vecs = head_dim >> 3;                        // uint4 per head
  const int units_per_row = (kLayout == BA_ROPE_ADJACENT) ? row_vecs : (row_vecs >> 1);
  const int total_rows = min(n_rows, __ldg(cu + n_blocks));
  const int row_step = blockDim.x / units_per_row;            // blockDim.x is a multiple of units_per_row
  const int u = threadIdx.x % units_per_row;
  const int row0 = blockIdx.x * (row_step * kRows) + threadIdx.x / units_per_row;

  // column of this thread's vector(s) inside the row, and its first rotary pair
  int vec_x, vec_y, m0;
  if (kLayout == BA_ROPE_ADJACENT) {
    vec_x = u; vec_y = u;
    m0 = (u % head_vecs) * 4;
  } else {
    int hv = head_vecs >> 1;                                  // vectors per half head
    int head = u / hv, v = u - head * hv;
    vec_x = head * head_vecs + v;
    vec_y = vec_x + hv;
    m0 = v * 8;
  }

  uint4 x[kRows], y[kRows];
  int blk[kRows];
  bool live[kRows];
  // Rows of a thread are close together, so they usually share a block: the block of a row is
  // looked up again only when the row leaves [c_begin, c_end).
  int c = 0, c_begin = 0, c_end = -1;
  long long shift = 0;                                        // source row = row + shift
#pragma unroll
  for (int i = 0; i < kRows; ++i) {
    const int r = row0 + i * row_step;
    live[i] = r < total_rows;
    blk[i] = 0;
    if (live[i]) {
      if (r < c_begin || r >= c_end) {
        c = upper_bound_i32(cu, n_blocks + 1, r) - 1;
        c = min(max(c, 0), n_blocks - 1);
        c_begin = __ldg(cu + c);
        c_end = __ldg(cu + c + 1);
        shift = src_off ? (long long)__ldg(src_off + c) - c_begin : 0;
      }
      blk[i] = c;
      const long long sr = r + shift;
      if (sr < 0 || sr >= n_src_rows) {
        ba_record_status(status, BA_ERR_INVALID_ARG);
        live[i] = false;
      } else {
        const uint4 *p = src + sr * row_vecs;
        x[i] = p[vec_x];
        if (kLayout == BA_ROPE_HALF) y[i] = p[vec_y];
      }
    }
  }
  // (cos, sin) of this thread's rotary pairs, reloaded only when the block changes
  int t_blk = -1, t_delta = 0;
  float4 tcs[4];
#pragma unroll
  for (int i = 0; i < kRows; ++i) {
    if (!live[i]) continue;
    int r = row0 + i * row_step;
    uint4 *q = dst + (long long)r * row_vecs;
    if (blk[i] != t_blk) {
      t_blk = blk[i];
      t_delta = __ldg(delta + t_blk);
      const float4 *t4 = reinterpret_cast<const float4 *>(table + t_blk * half_dim + m0);
      tcs[0] = __ldg(t4); tcs[1] = __ldg(t4 + 1);
      if (kLayout == BA_ROPE_HALF) { tcs[2] = __ldg(t4 + 2); tcs[3] = __ldg(t4 + 3); }
    }
    if (t_delta == 0) {                          // identity: copy bit-exactly
      q[vec_x] = x[i];
      if (kLayout == BA_ROPE_HALF) q[vec_y] = y[i];
      continue;
    }
    if (kLayout == BA_ROPE_ADJACENT) {
      const float4 a = tcs[0], b = tcs[1];                      // two (cos,sin) pairs per float4
      uint32_t w[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
      float2 cs[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y), make_float2(b.z, b.w)};
      uint32_t o[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float xo, yo;
        rot2(bf16_lo(w[j]), bf16_hi(w[j]), cs[j], xo, yo);
        o[j] = pack_bf16x2(xo, yo);
      }
      q[vec_x] = make_uint4(o[0], o[1], o[2], o[3]);
    } else {
      uint32_t wx[4] = {x[i].x, x[i].y, x[i].z, x[i].w};
      uint32_t wy[4] = {y[i].x, y[i].y, y[i].z, y[i].w};
      uint32_t ox[4], oy[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 cs = tcs[j];                             // pairs m0+2j, m0+2j+1
        float x0, y0, x1, y1;
        rot2(bf16_lo(wx[j]), bf16_lo(wy[j]), make_float2(cs.x, cs.y), x0, y0);
        rot2(bf16_hi(wx[j]), bf16_hi(wy[j]), make_float2(cs.z, cs.w), x1, y1);
        ox[j] = pack_bf16x2(x0, x1);
        oy[j] = pack_bf16x2(y0, y1);
      }
      q[vec_x] = make_uint4(ox[0], ox[1], ox[2], ox[3]);
      q[vec_y] = make_uint4(oy[0], oy[1], oy[2], oy[3]);
    }
  }
}

}  // namespace

ba_status ba_reencode_launch(ba_ctx *ctx, const void *k_src, const int32_t *src_off,
                             int32_t n_src_rows, void *k_dst, const int32_t *cu,
                             const int32_t *delta, int32_t n_blocks, int32_t n_rows, float2 *table,
                             cudaStream_t stream) {
  const int D = ctx->cfg.head_dim, H = ctx->cfg.n_kv_heads;
  const int half = D / 2;
  const double k = -2.0 / (double)D * log2(ctx->cfg.rope_theta);
  int n = n_blocks * half;
  ba_rope_table_kernel<<<(n + 127) / 128, 128, 0, stream>>>(delta, n_blocks, half, k, table);
  BA_CUDA_TRY(cudaGetLastError());

#ifndef BA_REENCODE_ROWS
#define BA_REENCODE_ROWS 2
#endif
  constexpr int kRows = BA_REENCODE_ROWS;   // rows in flight per thread
  const int row_vecs = H * D / 8;
  const bool adjacent = ctx->cfg.rope_layout == BA_ROPE_ADJACENT;
  const int units = adjacent ? row_vecs : row_vecs / 2;
  // threads per CTA: a multiple of the units per row, close to 256
  int threads = units >= 256 ? units : (256 / units) * units;
  if (threads > 512) return BA_ERR_UNSUPPORTED;   // more than 4096 bf16 per row
  const int rows_per_cta = (threads / units) * kRows;
  const int grid = (n_rows + rows_per_cta - 1) / rows_per_cta;
  if (adjacent)
    ba_reencode_kernel<BA_ROPE_ADJACENT, kRows><<<grid, threads, 0, stream>>>(
        (const uint4 *)k_src, (uint4 *)k_dst, src_off, n_src_rows, cu, delta, n_blocks, n_rows, D,
        row_vecs, table, ctx->dev_status);
  else
    ba_reencode_kernel<BA_ROPE_HALF, kRows><<<grid, threads, 0, stream>>>(
        (const uint4 *)k_src, (uint4 *)k_dst, src_off, n_src_rows, cu, delta, n_blocks, n_rows, D,
        row_vecs, table, ctx->dev_status);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 2;
  return BA_OK;
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
  return ba_reencode_launch(&tmp, k_src, src_off, n_src_rows, k_dst, cu, delta, n_blocks, n_rows,
                            g_noalloc_table[device], (cudaStream_t)stream);
}

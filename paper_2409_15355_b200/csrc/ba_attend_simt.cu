// Scalar (CUDA-core) attention under the Block-attention mask: one warp per
// (query row, query head), lanes striding over the visible keys with a private
// online softmax that is merged across the warp at the end.  It is the
// simplest device-side statement of the mask rules (Section 1, Section 2.4,
// Section 2.5 step 3) and serves shapes the tensor-core kernel does not take.
#include "ba_common.cuh"

namespace {

__device__ __forceinline__ int upper_bound_g(const int32_t *a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(a + mid) <= x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

template <int D>
struct LaneState {
  float m, l;
  float acc[D];
};

// Consume keys [begin, end) of (kbase, vbase) for one lane.  v_row(j) maps a key row to its value row.
template <int D, class VRow>
__device__ __forceinline__ void consume(LaneState<D> &st, const float *q_s, const __nv_bfloat16 *kbase,
                                        const __nv_bfloat16 *vbase, int kv_stride, int begin, int end,
                                        int lane, float scale, VRow v_row) {
  for (int j = begin + lane; j < end; j += 32) {
    const uint4 *kr = reinterpret_cast<const uint4 *>(kbase + (size_t)j * kv_stride);
    float s = 0.f;
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
      uint4 w = __ldg(kr + c);
      uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        s = fmaf(q_s[c * 8 + 2 * e], __uint_as_float(ww[e] << 16), s);
        s = fmaf(q_s[c * 8 + 2 * e + 1], __uint_as_float(ww[e] & 0xffff0000u), s);
      }
    }
    s *= scale;
    float m_new = fmaxf(st.m, s);
    float alpha = expf(st.m - m_new);   // exp(-inf) = 0 on the first key
    float p = expf(s - m_new);
    st.l = st.l * alpha + p;
    st.m = m_new;
    const uint4 *vr = reinterpret_cast<const uint4 *>(vbase + (size_t)v_row(j) * kv_stride);
#pragma unroll
    for (int c = 0; c < D / 8; ++c) {
      uint4 w = __ldg(vr + c);
      uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        st.acc[c * 8 + 2 * e] = fmaf(p, __uint_as_float(ww[e] << 16), st.acc[c * 8 + 2 * e] * alpha);
        st.acc[c * 8 + 2 * e + 1] = fmaf(p, __uint_as_float(ww[e] & 0xffff0000u), st.acc[c * 8 + 2 * e + 1] * alpha);
      }
    }
  }
}

template <int D>
__global__ void __launch_bounds__(128)
ba_attend_simt_kernel(ba_attend_args a, ba_segments seg, int Hq, int Hkv, float scale) {
  __shared__ float q_smem[4][D];
  if (__ldg(seg.totals + 7) != BA_TABLES_VALID) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long item = (long long)blockIdx.x * 4 + warp;
  const int row = (int)(item / Hq), h = (int)(item % Hq);
  if (row >= a.n_q_rows) return;
  const int G = Hq / Hkv, g = h / G;
  const int kv_stride = Hkv * D;

  float *q_s = q_smem[warp];
  const __nv_bfloat16 *qr = a.q + ((size_t)row * Hq + h) * D;
  for (int c = lane; c < D; c += 32) q_s[c] = __bfloat162float(qr[c]);
  __syncwarp();

  LaneState<D> st;
  st.m = -INFINITY; st.l = 0.f;
#pragma unroll
  for (int c = 0; c < D; ++c) st.acc[c] = 0.f;

  if (!a.final_only) {
    if (row >= seg.n_tokens) return;
    int b = __ldg(seg.tok_block + row);
    int begin = __ldg(seg.block_kv_begin + b);
    consume<D>(st, q_s, a.k + g * D, a.v + g * D, kv_stride, begin, row + 1, lane, scale,
               [](int j) { return j; });
  } else {
    int s = upper_bound_g(seg.cu_final_seq, seg.batch + 1, row) - 1;
    if (s < 0 || s >= seg.batch) return;
    int c0 = __ldg(seg.cu_cache_seq + s), c1 = __ldg(seg.cu_cache_seq + s + 1);
    c1 = min(c1, a.n_cache_rows);
    if (a.v_src_off) {
      const int32_t *cache_cu = seg.cache_cu;
      const int32_t *off = a.v_src_off;
      const int nbc = seg.n_cached_blocks, nv = a.n_v_rows;
      consume<D>(st, q_s, a.k_cache + g * D, a.v_cache + g * D, kv_stride, c0, c1, lane, scale,
                 [=](int j) {
                   int c = upper_bound_g(cache_cu, nbc + 1, j) - 1;
                   int r = __ldg(off + c) + (j - __ldg(cache_cu + c));
                   return min(max(r, 0), nv - 1);
                 });
    } else {
      consume<D>(st, q_s, a.k_cache + g * D, a.v_cache + g * D, kv_stride, c0, c1, lane, scale,
                 [](int j) { return j; });
    }
    int f0 = __ldg(seg.cu_final_seq + s);
    consume<D>(st, q_s, a.k + g * D, a.v + g * D, kv_stride, f0, row + 1, lane, scale,
               [](int j) { return j; });
  }

  // merge the 32 private softmax states
  float m_all = st.m;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xffffffffu, m_all, d));
  float w = expf(st.m - m_all);
  float l_all = st.l * w;
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) l_all += __shfl_xor_sync(0xffffffffu, l_all, d);
  float inv = 1.f / l_all;
  float *o32 = reinterpret_cast<float *>(a.o) + ((size_t)row * Hq + h) * D;
  __nv_bfloat16 *o16 = reinterpret_cast<__nv_bfloat16 *>(a.o) + ((size_t)row * Hq + h) * D;
#pragma unroll
  for (int c = 0; c < D; ++c) {
    float x = st.acc[c] * w;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) x += __shfl_xor_sync(0xffffffffu, x, d);
    if (lane == (c & 31)) {
      if (a.out_f32) o32[c] = x * inv; else o16[c] = __float2bfloat16_rn(x * inv);
    }
  }
  if (a.lse && lane == 0) a.lse[(size_t)row * Hq + h] = m_all + logf(l_all);
}

}  // namespace

ba_status ba_attend_simt_launch(ba_ctx *ctx, const ba_attend_args &a, const ba_segments *seg,
                                cudaStream_t stream) {
  const int Hq = ctx->cfg.n_q_heads, Hkv = ctx->cfg.n_kv_heads;
  long long items = (long long)a.n_q_rows * Hq;
  if (items == 0) return BA_OK;
  unsigned grid = (unsigned)((items + 3) / 4);
  if (ctx->cfg.head_dim == 128)
    ba_attend_simt_kernel<128><<<grid, 128, 0, stream>>>(a, *seg, Hq, Hkv, ctx->scale);
  else
    ba_attend_simt_kernel<64><<<grid, 128, 0, stream>>>(a, *seg, Hq, Hkv, ctx->scale);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 1;
  return BA_OK;
}

// Device-side core of the position re-encoding (Section 2.3, Eq. 1-3 collapsed into one rotation
// by the block's position delta), shared by the stand-alone kernel and by the attention kernel,
// whose two spare warps can carry a re-encoding job along in the background.
#pragma once

#include "ba_common.cuh"

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
// HALF layout: the vector at column c (< d/2) pairs with the vector at c + d/2, a thread moves both.
// A thread owns unit `u` (one vector column, or one column pair) and walks down the rows; what it
// knows about the block it is in -- bounds, source shift, delta, its (cos, sin) values -- stays in
// registers from one row to the next and is looked up again only when a row leaves the block.
// The source rows are read once: streaming loads keep them from displacing the re-encoded keys,
// which the attention launch that follows reads, in L2.
struct ba_reencode_state {
  int vec_x, vec_y, m0;              // the thread's vector column(s) and first rotary pair
  int c, c_begin, c_end;             // block of the last row and its row range
  long long shift;                   // source row = row + shift (contiguous source)
  int page0;                         // first entry of the block's page list (paged source)
  int t_blk, t_delta;                // block whose (cos, sin) values are loaded, and its delta
  float4 tcs[4];
};

template <int kLayout>
__device__ __forceinline__ void ba_reencode_state_init(const ba_reencode_job &job, int u, ba_reencode_state &st) {
  const int head_vecs = job.head_dim >> 3;                    // uint4 per head: 8 or 16
  if (kLayout == BA_ROPE_ADJACENT) {
    st.vec_x = u; st.vec_y = u;
    st.m0 = (u & (head_vecs - 1)) * 4;
  } else {
    const int hv = head_vecs >> 1;                            // vectors per half head: 4 or 8
    const int head = u / hv, v = u & (hv - 1);
    st.vec_x = head * head_vecs + v;
    st.vec_y = st.vec_x + hv;
    st.m0 = v * 8;
  }
  st.c = 0; st.c_begin = 0; st.c_end = -1; st.shift = 0; st.page0 = 0;
  st.t_blk = -1; st.t_delta = 0;
}

// Rows row0, row0 + row_step, ... (kRows of them, those below total_rows), all loads first.
template <int kLayout, int kRows>
__device__ __forceinline__ void ba_reencode_rows(const ba_reencode_job &job, ba_reencode_state &st, int row0,
                                                 int row_step, int total_rows, int32_t *status) {
  const uint4 *src = job.src;
  uint4 *dst = job.dst;
  const int32_t *src_off = job.src_off, *cu = job.cu;
  const int n_src_rows = job.n_src_rows, n_blocks = job.n_blocks, row_vecs = job.row_vecs;
  const int half_dim = job.head_dim >> 1;
  const int vec_x = st.vec_x, vec_y = st.vec_y;

  uint4 x[kRows], y[kRows];
  int blk[kRows];
  bool live[kRows];
#pragma unroll
  for (int i = 0; i < kRows; ++i) {
    const int r = row0 + i * row_step;
    live[i] = r < total_rows;
    blk[i] = 0;
    if (live[i]) {
      if (r < st.c_begin || r >= st.c_end) {
        int c;
        if (r >= st.c_end && st.c + 2 <= n_blocks && r < __ldg(cu + st.c + 2)) {
          c = st.c + 1;                                       // the usual case: the next block
        } else {
          c = upper_bound_i32(cu, n_blocks + 1, r) - 1;
          c = min(max(c, 0), n_blocks - 1);
        }
        st.c = c;
        st.c_begin = __ldg(cu + c);
        st.c_end = __ldg(cu + c + 1);
        st.shift = src_off ? (long long)__ldg(src_off + c) - st.c_begin : 0;
        st.page0 = job.page_cu ? __ldg(job.page_cu + c) : 0;
      }
      blk[i] = st.c;
      long long sr = r + st.shift;
      if (job.page_cu) {
        const int t = r - st.c_begin;
        const int page = __ldg(job.page_idx + st.page0 + (t >> job.page_lg));
        sr = page < 0 ? -1 : ((long long)page << job.page_lg) + (t & ((1 << job.page_lg) - 1));
      }
      if (sr < 0 || sr >= n_src_rows) {
        ba_record_status(status, BA_ERR_INVALID_ARG);
        live[i] = false;
      } else {
        const uint4 *p = src + sr * row_vecs;
        x[i] = __ldcs(p + vec_x);
        if (kLayout == BA_ROPE_HALF) y[i] = __ldcs(p + vec_y);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kRows; ++i) {
    if (!live[i]) continue;
    const int r = row0 + i * row_step;
    uint4 *q = dst + (long long)r * row_vecs;
    if (blk[i] != st.t_blk) {                    // (cos, sin) of this thread's rotary pairs in the new block
      st.t_blk = blk[i];
      st.t_delta = __ldg(job.delta + st.t_blk);
      const float4 *t4 = reinterpret_cast<const float4 *>(job.table + st.t_blk * half_dim + st.m0);
      st.tcs[0] = __ldg(t4); st.tcs[1] = __ldg(t4 + 1);
      if (kLayout == BA_ROPE_HALF) { st.tcs[2] = __ldg(t4 + 2); st.tcs[3] = __ldg(t4 + 3); }
    }
    if (st.t_delta == 0) {                       // identity: copy bit-exactly
      q[vec_x] = x[i];
      if (kLayout == BA_ROPE_HALF) q[vec_y] = y[i];
      continue;
    }
    if (kLayout == BA_ROPE_ADJACENT) {
      const float4 a = st.tcs[0], b = st.tcs[1];              // two (cos,sin) pairs per float4
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
        const float4 cs = st.tcs[j];                          // pairs m0+2j, m0+2j+1
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

// ---------------------------------------------------------------------------------------------
// Background engine for one warp of another kernel.  Chunks of up to `rows_per_chunk` rows are
// drawn from a device-wide counter, their source rows are fetched into shared memory with bulk
// asynchronous copies (two chunks in flight per warp, no registers tied up), rotated and written
// to the destination with coalesced 16-byte stores.  Any number of warps on any number of SMs may
// run it concurrently on the same job; together they finish it.
// ---------------------------------------------------------------------------------------------
struct ba_bg_smem {
  uint64_t bar[2];          // one per stage: bytes of the chunk have landed
  int blk[2][32];           // block of every row of the chunk (-1: row skipped)
  int chunk[2];
};

__device__ __forceinline__ void ba_bulk_load(void *dst_smem, const void *src, uint32_t bytes, uint64_t *bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"((uint32_t)__cvta_generic_to_shared(dst_smem)), "l"(src), "r"(bytes),
                 "r"((uint32_t)__cvta_generic_to_shared(bar))
               : "memory");
}

// `wait` is the caller's bounded mbarrier wait: bool wait(uint64_t *bar, uint32_t parity).
// `stage_buf` points to 2 * rows_per_chunk * row_bytes bytes of 16-byte aligned shared memory owned
// by this warp; `sm` to its ba_bg_smem (barriers initialised with count 1 by the caller).
template <class Wait>
__device__ __forceinline__ void ba_reencode_background(const ba_reencode_job &job, int32_t *chunk_counter,
                                                       uint8_t *stage_buf, ba_bg_smem *sm, int rows_per_chunk,
                                                       int32_t *status, Wait wait) {
  const int lane = threadIdx.x & 31;
  const int row_vecs = job.row_vecs, half_dim = job.head_dim >> 1, head_vecs = job.head_dim >> 3;
  const uint32_t row_bytes = (uint32_t)row_vecs * 16u;
  const int total_rows = min(job.n_rows, __ldg(job.cu + job.n_blocks));
  const int n_chunks = (total_rows + rows_per_chunk - 1) / rows_per_chunk;
  const bool adjacent = job.layout == BA_ROPE_ADJACENT;
  if (job.gen && __ldg(job.gen) != job.gen_expected) {     // the rotation table is not the one this job was given
    if (lane == 0) ba_record_status(status, BA_ERR_INVALID_ARG);
    return;
  }

  // fetch: draw a chunk, resolve its rows, start the copies into stage `s`; returns false when the job is exhausted
  auto fetch = [&](int s) -> bool {
    int chunk = 0;
    if (lane == 0) chunk = atomicAdd(chunk_counter, 1);
    chunk = __shfl_sync(0xffffffffu, chunk, 0);
    if (lane == 0) sm->chunk[s] = chunk;
    if (chunk >= n_chunks) return false;
    const int r = chunk * rows_per_chunk + lane;
    long long sr = -1;
    int c = -1;
    if (lane < rows_per_chunk && r < total_rows) {
      c = upper_bound_i32(job.cu, job.n_blocks + 1, r) - 1;
      c = min(max(c, 0), job.n_blocks - 1);
      const int c_begin = __ldg(job.cu + c);
      sr = ba_job_source_row(job, c, c_begin, r - c_begin);
      if (sr < 0 || sr >= job.n_src_rows) { ba_record_status(status, BA_ERR_INVALID_ARG); sr = -1; c = -1; }
    }
    if (lane < 32) sm->blk[s][lane] = c;
    const unsigned live = __ballot_sync(0xffffffffu, sr >= 0);
    if (lane == 0) {
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                   ::"r"((uint32_t)__cvta_generic_to_shared(&sm->bar[s])), "r"((uint32_t)__popc(live) * row_bytes)
                   : "memory");
    }
    __syncwarp();
    if (sr >= 0)
      ba_bulk_load(stage_buf + ((size_t)s * rows_per_chunk + lane) * row_bytes,
                   reinterpret_cast<const uint8_t *>(job.src) + (size_t)sr * row_bytes, row_bytes, &sm->bar[s]);
    return true;
  };

  bool have[2];
  uint32_t phase[2] = {0u, 0u};
  have[0] = fetch(0);
  have[1] = have[0] ? fetch(1) : false;
  for (int s = 0; have[s]; s ^= 1) {
    if (!wait(&sm->bar[s], phase[s])) return;
    phase[s] ^= 1u;
    __syncwarp();
    const int chunk = sm->chunk[s];
    const uint4 *buf = reinterpret_cast<const uint4 *>(stage_buf + (size_t)s * rows_per_chunk * row_bytes);
    const int units_per_row = adjacent ? row_vecs : (row_vecs >> 1);
    const int n_units = rows_per_chunk * units_per_row;
    for (int idx = lane; idx < n_units; idx += 32) {
      const int i = idx / units_per_row, u = idx - i * units_per_row;
      const int c = sm->blk[s][i];
      if (c < 0) continue;
      const int r = chunk * rows_per_chunk + i;
      uint4 *q = job.dst + (size_t)r * row_vecs;
      const uint4 *row = buf + (size_t)i * row_vecs;
      const int dlt = __ldg(job.delta + c);
      if (adjacent) {
        const uint4 x = row[u];
        if (dlt == 0) { q[u] = x; continue; }
        const float4 *t4 = reinterpret_cast<const float4 *>(job.table + c * half_dim + (u % head_vecs) * 4);
        const float4 a = __ldg(t4), b = __ldg(t4 + 1);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
        const float2 cs[4] = {make_float2(a.x, a.y), make_float2(a.z, a.w), make_float2(b.x, b.y), make_float2(b.z, b.w)};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float xo, yo;
          rot2(bf16_lo(w[j]), bf16_hi(w[j]), cs[j], xo, yo);
          o[j] = pack_bf16x2(xo, yo);
        }
        q[u] = make_uint4(o[0], o[1], o[2], o[3]);
      } else {
        const int hv = head_vecs >> 1;
        const int head = u / hv, v = u - head * hv;
        const int vec_x = head * head_vecs + v, vec_y = vec_x + hv;
        const uint4 x = row[vec_x], y = row[vec_y];
        if (dlt == 0) { q[vec_x] = x; q[vec_y] = y; continue; }
        const float4 *t4 = reinterpret_cast<const float4 *>(job.table + c * half_dim + v * 8);
        const uint32_t wx[4] = {x.x, x.y, x.z, x.w}, wy[4] = {y.x, y.y, y.z, y.w};
        uint32_t ox[4], oy[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float4 cs = __ldg(t4 + j);
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
    __syncwarp();                 // the stage is free again
    have[s] = fetch(s);
  }
}


// Backward pass of attention under the Block-attention mask for sm_100a (Section 2.4: block
// fine-tuning trains with this mask in place of the lower-triangular one, so the gradients flow
// through the same masked softmax as ba_block_prefill).
//
// With P = softmax(scale Q K^T + mask), O = P V and delta_i = dO_i . O_i:
//     dV = P^T dO,   dP = dO V^T,   dS = P * (dP - delta),   dQ = scale dS K,   dK = scale dS^T Q.
// P is recomputed from the log-sum-exp the forward pass stored.  Two kernels, both built from
// 128 x 128 tiles on the tensor cores (tcgen05.mma, accumulators in tensor memory), neither uses
// atomics, so results are run-to-run identical:
//   * ba_bwd_dkv_kernel: one CTA owns 128 keys of one block and one KV head and walks over every
//     query tile that sees them (all heads of the group).  It forms the scores transposed, S^T = K Q^T
//     and dP^T = V dO^T (keys on the tensor-memory lanes, query rows on the columns), so that its 128
//     threads -- one per key -- write P^T and dS^T back to tensor memory as bf16, where they are the A
//     operands of dV += P^T dO and dK += dS^T Q (nothing goes through shared memory, nothing is transposed).
//   * ba_bwd_dq_kernel: one CTA owns one query tile (tokens x heads of one KV group, as in the
//     forward kernel) and walks over the key tiles it sees: S = Q K^T, dP = dO V^T (query rows on the
//     lanes), dS written to tensor memory, dQ += dS K.
// The tiles a CTA walks over (Q and dO there, K and V here) are double-buffered in shared memory, so the
// loads of the next tile run under the current one.  Both kernels work in steps of 64 columns of S and dP with
// two buffers of each in tensor memory (2 x 2 x 64 columns beside the accumulators): while the threads turn
// one step's scores into P and dS, the tensor core forms the next step's scores and multiplies the previous
// step's P and dS.
#include <math.h>

#include "ba_common.cuh"
#include "ba_sm100.cuh"

using namespace sm100;

int ba_heads_per_tile(const ba_config &c);

namespace {

// warps 0-7: two threads per tile row (tensor-memory lane = tid & 127), warps w and w + 4 share a lane quarter and
// take one half of every step's 64 columns each, so that every SM sub-partition has two warps to hide the
// latency of tensor-memory loads, shared-memory reads and exponentials; warp 8: loads and MMA issue
constexpr int kBwdThreads = 288;
constexpr int kRowThreads = 256;
constexpr int kCtlWarp = 8;
constexpr int kTile = 128;

struct BwdParams {
  const float *lse;          // [T, Hq] natural-log softmax denominators of the forward pass
  const float *delta;        // [T, Hq] dO . O
  void *dq, *dk, *dv;
  int out_f32;
  int32_t *status;
  int Hq, Hkv, G, hpt, hpt_log2, tok;
  float scale, scale_log2;
  int mode;
  int n_rows;                // T
  ba_segments seg;
};

template <int D>
struct BwdLayout {
  static constexpr int kChunks = D / 64;
  static constexpr int kRegion = 128 * 128;              // 128 rows x 128 bytes
  static constexpr int kTileBytes = 128 * D * 2;
  // two tiles that stay for the whole CTA (K, V in the dK/dV kernel; Q, dO in the dQ kernel) and two
  // buffers of two tiles each for the ones it walks over
  static constexpr int kFix0 = 0, kFix1 = kTileBytes;
  static constexpr int kWalk = 2 * kTileBytes;            // buffer b: tiles at kWalk + b * 2 * kTileBytes, + kTileBytes
  static constexpr int kStats = 6 * kTileBytes;           // dK/dV kernel: per query row lse * log2 e, dO . O * scale, visible keys; two buffers of each
  static constexpr int kCtrl = kStats + 2 * 128 * 16;
  static constexpr int kBytes = kCtrl + 256;
};

struct BwdCtrl {
  uint64_t fix_full, walk_full[2], walk_free[2];
  uint64_t sd_full[2], rows_done[2];     // per buffer of S / dP in tensor memory
  uint64_t fin;                          // every product of the CTA has completed
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void named_barrier_rows() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

__device__ __forceinline__ int upper_bound_dev(const int32_t *a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(a + mid) <= x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// The kernels work in steps of 64 columns of S and dP: tensor memory then holds two buffers of each next to the
// accumulators, so the threads turn one step's scores into P / dS while the tensor core forms the next step's
// scores and multiplies the previous step's P / dS.
//
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
  uint64_t d;
  asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}

// The arithmetic of both helpers is packed fp32x2: for a pair of columns, x = s * scale_log2 - lse_log2 (one FMA),
// p = exp2(x) (two), t = dp * scale - delta * scale (one FMA), ds = p * t (one multiply).  kMasked = false is for
// steps in which every (row, key) pair is visible: no comparison at all.
//
// dQ kernel, one query row (= lane) against 64 keys: the thread takes chunk `c` (32 columns) of the step's S and
// dP and writes dS back over the first 16 dP columns it has read, as bf16 (two per column): the A operand of
// dQ += dS K.  `n_ok`: columns 0 .. n_ok - 1 of the step are visible to this row (0: none).
template <bool kMasked>
__device__ __forceinline__ void bwd_row_ds(uint32_t tS, uint32_t tDP, int c, int n_ok, float scale_log2, float lse_log2,
                                           float delta_scaled, float scale) {
  uint32_t s[32], dp[32];
  tmem_ld_32x32b_x32(tS + c * 32, s);
  tmem_ld_32x32b_x32(tDP + c * 32, dp);
  tmem_wait_ld();
  const uint64_t sl2 = pack2(scale_log2, scale_log2), nl2 = pack2(-lse_log2, -lse_log2);
  const uint64_t sc2 = pack2(scale, scale), nd2 = pack2(-delta_scaled, -delta_scaled);
  uint32_t dw[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const uint64_t x2 = fma2(pack2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), sl2, nl2);
    float x0, x1;
    unpack2(x2, x0, x1);
    float p0 = ex2(x0), p1 = ex2(x1);
    if (kMasked) {
      const int e0 = c * 32 + 2 * i;
      if (e0 >= n_ok) p0 = 0.f;
      if (e0 + 1 >= n_ok) p1 = 0.f;
    }
    const uint64_t t2 = fma2(pack2(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])), sc2, nd2);
    float d0, d1;
    unpack2(mul2(pack2(p0, p1), t2), d0, d1);
    __nv_bfloat162 dv = __floats2bfloat162_rn(d0, d1);
    dw[i] = *reinterpret_cast<uint32_t *>(&dv);
  }
  tmem_st16(tDP + c * 32, dw);
  tmem_wait_st();
}

// dK/dV kernel, one key (= lane `j`) against 64 query rows of a tile (= columns): the thread takes chunk `c`
// (32 columns) of the step's S^T and dP^T; the per-row values -- lse * log2 e, dO . O * scale, and the number of
// keys of this tile the row sees -- are read from shared memory, the same address by every thread.  P^T goes back
// over the S^T columns and dS^T over the dP^T columns as bf16 -- each thread over columns it has read itself,
// because the other thread of the lane works on its own 32 columns at its own pace.
template <bool kMasked>
__device__ __forceinline__ void bwd_key_p_ds(uint32_t tST, uint32_t tDPT, int c, int j, const float *lse2, const float *dls,
                                             const int *lim, float scale_log2, float scale) {
  uint32_t s[32], dp[32];
  tmem_ld_32x32b_x32(tST + c * 32, s);
  tmem_ld_32x32b_x32(tDPT + c * 32, dp);
  tmem_wait_ld();
  const uint64_t sl2 = pack2(scale_log2, scale_log2), sc2 = pack2(scale, scale);
  uint32_t pw[16], dw[16];
#pragma unroll
  for (int q = 0; q < 8; ++q) {                          // four columns at a time: one 16-byte read of each per-row array
    const float4 l4 = *reinterpret_cast<const float4 *>(lse2 + c * 32 + 4 * q);
    const float4 d4 = *reinterpret_cast<const float4 *>(dls + c * 32 + 4 * q);
    int4 m4 = make_int4(0, 0, 0, 0);
    if (kMasked) m4 = *reinterpret_cast<const int4 *>(lim + c * 32 + 4 * q);
#pragma unroll
    for (int e = 0; e < 2; ++e) {
      const int i = 2 * q + e;
      const uint64_t nl2 = e ? pack2(-l4.z, -l4.w) : pack2(-l4.x, -l4.y);
      const uint64_t nd2 = e ? pack2(-d4.z, -d4.w) : pack2(-d4.x, -d4.y);
      const uint64_t x2 = fma2(pack2(__uint_as_float(s[2 * i]), __uint_as_float(s[2 * i + 1])), sl2, nl2);
      float x0, x1;
      unpack2(x2, x0, x1);
      float p0 = ex2(x0), p1 = ex2(x1);
      if (kMasked) {
        if (j >= (e ? m4.z : m4.x)) p0 = 0.f;
        if (j >= (e ? m4.w : m4.y)) p1 = 0.f;
      }
      const uint64_t t2 = fma2(pack2(__uint_as_float(dp[2 * i]), __uint_as_float(dp[2 * i + 1])), sc2, nd2);
      float d0, d1;
      unpack2(mul2(pack2(p0, p1), t2), d0, d1);
      __nv_bfloat162 pv = __floats2bfloat162_rn(p0, p1), dv = __floats2bfloat162_rn(d0, d1);
      pw[i] = *reinterpret_cast<uint32_t *>(&pv);
      dw[i] = *reinterpret_cast<uint32_t *>(&dv);
    }
  }
  tmem_st16(tST + c * 32, pw);
  tmem_st16(tDPT + c * 32, dw);
  tmem_wait_st();
}

// Writes one accumulator row (D fp32 columns of tensor memory, lane = row) to global memory.
// The two threads of a row take alternate chunks of 32 columns (`half` = 0 or 1).
template <int D>
__device__ __forceinline__ void store_acc_row(uint32_t tAcc, void *dst_base, size_t elem_off, int out_f32, bool valid,
                                              int half) {
#pragma unroll
  for (int cc = 0; cc < D / 64; ++cc) {
    const int c = 2 * cc + half;
    uint32_t a[32];
    tmem_ld_32x32b_x32(tAcc + c * 32, a);
    tmem_wait_ld();
    if (!valid) continue;
    if (out_f32) {
      float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(dst_base) + elem_off + c * 32);
#pragma unroll
      for (int i = 0; i < 8; ++i)
        dst[i] = make_float4(__uint_as_float(a[4 * i]), __uint_as_float(a[4 * i + 1]), __uint_as_float(a[4 * i + 2]),
                             __uint_as_float(a[4 * i + 3]));
    } else {
      uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(dst_base) + elem_off + c * 32);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        uint32_t w[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(a[8 * i + 2 * e]), __uint_as_float(a[8 * i + 2 * e + 1]));
          w[e] = *reinterpret_cast<uint32_t *>(&v);
        }
        dst[i] = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
  }
}

// ---------------------------------------------------------------------------------------------
// dK, dV: CTA = (128-key tile of one block, KV head)
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
ba_bwd_dkv_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                  const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                  const BwdParams p) {
  using L = BwdLayout<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  BwdCtrl *ctrl = reinterpret_cast<BwdCtrl *>(smem + L::kCtrl);
  const int tid = threadIdx.x, warp = tid >> 5;
  const ba_segments &sg = p.seg;
  if (__ldg(sg.totals + 7) != BA_TABLES_VALID) return;

  // which keys: tile `kt` of the batch (a tile never spans two blocks), KV head `g`
  const int kt = blockIdx.x, g = blockIdx.y;
  if (kt >= __ldg(sg.cu_ktile + sg.n_blocks)) return;
  const int b = upper_bound_dev(sg.cu_ktile, sg.n_blocks + 1, kt) - 1;
  const int blk0 = __ldg(sg.cu_block + b), blk1 = __ldg(sg.cu_block + b + 1);
  const int k0 = blk0 + (kt - __ldg(sg.cu_ktile + b)) * kTile;
  const int n_keys = min(kTile, blk1 - k0);
  // which queries see them: rows k0 .. end of the block (causally); in full mode the rest of the sequence
  // as well; in block mode the rows of the sequence's final block (they see every earlier block)
  const int sq = __ldg(sg.block_seq + b);
  const int seq1 = __ldg(sg.cu_seq + sq + 1);
  const int fin0 = __ldg(sg.cu_block + __ldg(sg.cu_seq_block + sq + 1) - 1);    // first row of the final block
  const bool is_final = __ldg(sg.block_is_final + b) != 0;
  const int r1_begin = k0, r1_end = (p.mode == BA_MODE_FULL) ? seq1 : blk1;     // causal range
  int r2_begin = 0, r2_end = 0;                                                 // range that sees all the keys
  if (p.mode == BA_MODE_BLOCK && !is_final) { r2_begin = fin0; r2_end = seq1; }
  const int tiles1 = (r1_end - r1_begin + p.tok - 1) / p.tok, tiles2 = (r2_end - r2_begin + p.tok - 1) / p.tok;
  const int n_chunks = p.G / p.hpt;                                             // head chunks of this KV group
  const int n_iter = (tiles1 + tiles2) * n_chunks;
  // iteration `it`: token tile it / n_chunks, head chunk it % n_chunks
  auto iter_rows = [&](int it, int &row0, int &row_end, bool &causal, int &head0) {
    const int ti = it / n_chunks, ch = it - ti * n_chunks;
    causal = ti < tiles1;
    row0 = causal ? r1_begin + ti * p.tok : r2_begin + (ti - tiles1) * p.tok;
    row_end = causal ? r1_end : r2_end;
    head0 = g * p.G + ch * p.hpt;
  };

  if (tid == 0) {
    mbar_init(&ctrl->fix_full, 1); mbar_init(&ctrl->fin, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&ctrl->walk_full[i], 1); mbar_init(&ctrl->walk_free[i], 1);
      mbar_init(&ctrl->sd_full[i], 1); mbar_init(&ctrl->rows_done[i], kRowThreads);
    }
    ctrl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kCtlWarp) { tmem_alloc(&ctrl->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctrl->tmem_base;
  volatile int *abort_flag = &ctrl->abort_flag;
  // tensor memory: S^T buffers at columns 0 and 64, dP^T buffers at 128 and 192 (64 query rows each), dV, dK
  const uint32_t tST = tmem, tDPT = tmem + 128, tDV = tmem + 256, tDK = tmem + 384;
  const int n_steps = 2 * n_iter;                        // step i: query rows 64 (i & 1) .. + 63 of tile i >> 1

  if (warp == kCtlWarp) {
    if (elect_one()) {
      constexpr uint32_t idesc_nt = make_idesc_bf16(128, 64, 0);                // both operands K-major, 64 query rows
      constexpr uint32_t idesc_tn = make_idesc_bf16(128, D, 1);                 // A from tensor memory, B MN-major
      const uint64_t k_desc = make_smem_desc(smem_u32(smem + L::kFix0), 16, 1024);
      const uint64_t v_desc = make_smem_desc(smem_u32(smem + L::kFix1), 16, 1024);
      bool ok = true;
      auto load_walk = [&](int it) {                     // Q and dO tiles of tile `it` into buffer it & 1
        int row0, row_end, head0; bool causal;
        iter_rows(it, row0, row_end, causal, head0);
        uint8_t *dst = smem + L::kWalk + (it & 1) * 2 * L::kTileBytes;
        mbar_arrive_expect_tx(&ctrl->walk_full[it & 1], 2 * L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c) {
          tma_load_3d(dst + c * L::kRegion, &tmap_q, &ctrl->walk_full[it & 1], c * 64, head0, row0);
          tma_load_3d(dst + L::kTileBytes + c * L::kRegion, &tmap_do, &ctrl->walk_full[it & 1], c * 64, head0, row0);
        }
      };
      // S^T = K Q^T and dP^T = V dO^T for the 64 query rows of step i.  They follow the gradient products of step
      // i - 2 (same buffers) on the tensor pipe in issue order, so those have read P^T and dS^T before.
      auto issue_scores = [&](int i) -> bool {
        const int it = i >> 1, h = i & 1;
        if (h == 0) {
          if (!mbar_wait(&ctrl->walk_full[it & 1], (it >> 1) & 1, abort_flag)) return false;
          tc_fence_after();
        }
        const uint32_t walk = smem_u32(smem + L::kWalk + (it & 1) * 2 * L::kTileBytes) + h * 64 * 128;   // rows 64 h ..
        const uint64_t q_desc = make_smem_desc(walk, 16, 1024);
        const uint64_t do_desc = make_smem_desc(walk + L::kTileBytes, 16, 1024);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tST + (i & 1) * 64, k_desc + off, q_desc + off, idesc_nt, k > 0);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tDPT + (i & 1) * 64, v_desc + off, do_desc + off, idesc_nt, k > 0);
        }
        mma_commit(&ctrl->sd_full[i & 1]);
        return true;
      };
      // dV += P^T dO, dK += dS^T Q over the 64 query rows of step i (16 at a time)
      auto issue_grads = [&](int i) -> bool {
        const int it = i >> 1, h = i & 1;
        if (!mbar_wait(&ctrl->rows_done[i & 1], (i >> 1) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint32_t walk = smem_u32(smem + L::kWalk + (it & 1) * 2 * L::kTileBytes);
        const uint64_t q_mn = make_smem_desc(walk, L::kRegion, 1024);
        const uint64_t do_mn = make_smem_desc(walk + L::kTileBytes, L::kRegion, 1024);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_ts(tDV, tST + (i & 1) * 64 + (k >> 1) * 32 + (k & 1) * 8, do_mn + (uint64_t)(((h * 64 + k * 16) * 128) >> 4), idesc_tn,
                 (i > 0 || k > 0) ? 1u : 0u);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_ts(tDK, tDPT + (i & 1) * 64 + (k >> 1) * 32 + (k & 1) * 8, q_mn + (uint64_t)(((h * 64 + k * 16) * 128) >> 4), idesc_tn,
                 (i > 0 || k > 0) ? 1u : 0u);
        if (h == 1) mma_commit(&ctrl->walk_free[it & 1]);   // the tile's Q and dO have been read for the last time
        return true;
      };
      mbar_arrive_expect_tx(&ctrl->fix_full, 2 * L::kTileBytes);
      for (int c = 0; c < L::kChunks; ++c) {
        tma_load_3d(smem + L::kFix0 + c * L::kRegion, &tmap_k, &ctrl->fix_full, c * 64, g, k0);
        tma_load_3d(smem + L::kFix1 + c * L::kRegion, &tmap_v, &ctrl->fix_full, c * 64, g, k0);
      }
      if (n_iter > 0) load_walk(0);
      if (n_iter > 1) load_walk(1);
      ok = mbar_wait(&ctrl->fix_full, 0, abort_flag);
      int reload = -1;                                   // tile whose buffer is refilled once its products have completed
      for (int i = 0; i <= n_steps && ok; ++i) {
        if (i < n_steps) ok = issue_scores(i);
        if (ok && reload >= 0) {
          if (reload + 2 < n_iter) {
            ok = mbar_wait(&ctrl->walk_free[reload & 1], (reload >> 1) & 1, abort_flag);
            if (ok) load_walk(reload + 2);
          }
          reload = -1;
        }
        if (ok && i > 0) {
          ok = issue_grads(i - 1);
          if ((i - 1) & 1) reload = (i - 1) >> 1;
        }
      }
      if (ok) mma_commit(&ctrl->fin);
    }
  } else {
    const int j = tid & 127;                             // key of the tile = tensor-memory lane
    const int ch = tid >> 7;                             // which 32 of a step's 64 columns this thread takes
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    // per query row of the tile, two buffers: lse * log2 e [128], dO . O * scale [128], visible keys [128]
    float *st_lse = reinterpret_cast<float *>(smem + L::kStats);
    float *st_dls = st_lse + 2 * 128;
    int *st_lim = reinterpret_cast<int *>(st_dls + 2 * 128);
    bool ok = true;
    for (int i = 0; i < n_steps; ++i) {
      const int it = i >> 1, h = i & 1;
      int row0, row_end, head0; bool causal;
      iter_rows(it, row0, row_end, causal, head0);
      if (h == 0) {
        if (tid < 128) {
          // this thread also prepares what every key thread needs to know about query row `tid` of the tile
          const int tok_i = row0 + (tid >> p.hpt_log2);
          const int head = head0 + (tid & (p.hpt - 1));
          float l2 = 0.f, dl = 0.f; int lm = 0;
          if (tok_i < row_end) {
            l2 = __ldg(p.lse + (size_t)tok_i * p.Hq + head) * 1.4426950408889634f;
            dl = __ldg(p.delta + (size_t)tok_i * p.Hq + head) * p.scale;
            lm = causal ? max(0, min(n_keys, tok_i - k0 + 1)) : n_keys;      // keys 0 .. lm - 1 of the tile are visible
          }
          st_lse[(it & 1) * 128 + tid] = l2; st_dls[(it & 1) * 128 + tid] = dl; st_lim[(it & 1) * 128 + tid] = lm;
        }
        named_barrier_rows();
      }
      // every pair of this step visible?  (all 128 keys exist, the step's rows exist and, in the causal range,
      // already its first row sees the tile's last key)
      const int tok_first = row0 + ((h * 64) >> p.hpt_log2), tok_last = row0 + ((h * 64 + 63) >> p.hpt_log2);
      const bool all_visible = n_keys == kTile && tok_last < row_end && (!causal || tok_first - k0 + 1 >= kTile);
      ok = mbar_wait(&ctrl->sd_full[i & 1], (i >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const int so = (it & 1) * 128 + h * 64;
      if (all_visible)
        bwd_key_p_ds<false>(tST + (i & 1) * 64 + lane_off, tDPT + (i & 1) * 64 + lane_off, ch, j, st_lse + so, st_dls + so,
                            st_lim + so, p.scale_log2, p.scale);
      else
        bwd_key_p_ds<true>(tST + (i & 1) * 64 + lane_off, tDPT + (i & 1) * 64 + lane_off, ch, j, st_lse + so, st_dls + so,
                           st_lim + so, p.scale_log2, p.scale);
      tc_fence_before();
      mbar_arrive(&ctrl->rows_done[i & 1]);
    }
    // accumulators: lane = key row of the tile
    if (ok && n_iter > 0) ok = mbar_wait(&ctrl->fin, 0, abort_flag);
    if (ok && n_iter > 0) {
      tc_fence_after();
      const bool valid = j < n_keys;
      const size_t off = ((size_t)(k0 + j) * p.Hkv + g) * D;
      store_acc_row<D>(tDV + lane_off, p.dv, off, p.out_f32, valid, ch);
      store_acc_row<D>(tDK + lane_off, p.dk, off, p.out_f32, valid, ch);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && ctrl->abort_flag) ba_record_status(p.status, BA_ERR_TIMEOUT);
  if (warp == kCtlWarp) tmem_dealloc(tmem, 512);
}

// ---------------------------------------------------------------------------------------------
// dQ: CTA = (query tile of `tok` tokens x `hpt` heads, head chunk)
// ---------------------------------------------------------------------------------------------
template <int D>
__global__ void __launch_bounds__(kBwdThreads, 1)
ba_bwd_dq_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_do,
                 const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                 const BwdParams p) {
  using L = BwdLayout<D>;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  BwdCtrl *ctrl = reinterpret_cast<BwdCtrl *>(smem + L::kCtrl);
  const int tid = threadIdx.x, warp = tid >> 5;
  const ba_segments &sg = p.seg;
  if (__ldg(sg.totals + 7) != BA_TABLES_VALID) return;

  // query tile: half `blockIdx.x & 1` of query-tile pair `blockIdx.x >> 1` (the pairs of the forward kernel)
  const int pair = blockIdx.x >> 1, half = blockIdx.x & 1;
  if (pair >= __ldg(sg.totals + 2)) return;
  const int b = upper_bound_dev(sg.cu_qtile, sg.n_blocks + 1, pair) - 1;
  const int blk0 = __ldg(sg.cu_block + b), blk1 = __ldg(sg.cu_block + b + 1);
  const int q0 = blk0 + (pair - __ldg(sg.cu_qtile + b)) * 2 * p.tok + half * p.tok;
  if (q0 >= blk1) return;
  const int q_end = min(q0 + p.tok, blk1);                // rows q0 .. q_end - 1
  const int kv0 = __ldg(sg.block_kv_begin + b);           // row i sees keys kv0 .. i
  const int head0 = blockIdx.y * p.hpt, g = head0 / p.G;
  const int n_iter = (q_end - kv0 + kTile - 1) / kTile;   // key tiles kv0 + 128 j
  const int n_steps = (q_end - kv0 + 63) / 64;            // step i: keys kv0 + 64 i .. + 63 (half of tile i >> 1)

  if (tid == 0) {
    mbar_init(&ctrl->fix_full, 1); mbar_init(&ctrl->fin, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&ctrl->walk_full[i], 1); mbar_init(&ctrl->walk_free[i], 1);
      mbar_init(&ctrl->sd_full[i], 1); mbar_init(&ctrl->rows_done[i], kRowThreads);
    }
    ctrl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == kCtlWarp) { tmem_alloc(&ctrl->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctrl->tmem_base;
  volatile int *abort_flag = &ctrl->abort_flag;
  // tensor memory: S buffers at columns 0 and 64, dP buffers at 128 and 192 (64 keys each), dQ
  const uint32_t tS = tmem, tDP = tmem + 128, tDQ = tmem + 256;

  if (warp == kCtlWarp) {
    if (elect_one()) {
      constexpr uint32_t idesc_nt = make_idesc_bf16(128, 64, 0);
      constexpr uint32_t idesc_nn = make_idesc_bf16(128, D, 1);                 // A from tensor memory (dS), B MN-major (K)
      const uint64_t q_desc = make_smem_desc(smem_u32(smem + L::kFix0), 16, 1024);
      const uint64_t do_desc = make_smem_desc(smem_u32(smem + L::kFix1), 16, 1024);
      bool ok = true;
      auto load_walk = [&](int it) {                     // K and V tiles of key tile `it` into buffer it & 1
        uint8_t *dst = smem + L::kWalk + (it & 1) * 2 * L::kTileBytes;
        mbar_arrive_expect_tx(&ctrl->walk_full[it & 1], 2 * L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c) {
          tma_load_3d(dst + c * L::kRegion, &tmap_k, &ctrl->walk_full[it & 1], c * 64, g, kv0 + it * kTile);
          tma_load_3d(dst + L::kTileBytes + c * L::kRegion, &tmap_v, &ctrl->walk_full[it & 1], c * 64, g, kv0 + it * kTile);
        }
      };
      auto issue_scores = [&](int i) -> bool {           // S = Q K^T, dP = dO V^T for the 64 keys of step i
        const int it = i >> 1, h = i & 1;
        if (h == 0) {
          if (!mbar_wait(&ctrl->walk_full[it & 1], (it >> 1) & 1, abort_flag)) return false;
          tc_fence_after();
        }
        const uint32_t walk = smem_u32(smem + L::kWalk + (it & 1) * 2 * L::kTileBytes) + h * 64 * 128;   // keys 64 h ..
        const uint64_t k_desc = make_smem_desc(walk, 16, 1024);
        const uint64_t v_desc = make_smem_desc(walk + L::kTileBytes, 16, 1024);
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tS + (i & 1) * 64, q_desc + off, k_desc + off, idesc_nt, k > 0);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tDP + (i & 1) * 64, do_desc + off, v_desc + off, idesc_nt, k > 0);
        }
        mma_commit(&ctrl->sd_full[i & 1]);
        return true;
      };
      auto issue_grads = [&](int i) -> bool {            // dQ += dS K over the 64 keys of step i (16 at a time)
        const int it = i >> 1, h = i & 1;
        if (!mbar_wait(&ctrl->rows_done[i & 1], (i >> 1) & 1, abort_flag)) return false;
        tc_fence_after();
        const uint64_t k_mn = make_smem_desc(smem_u32(smem + L::kWalk + (it & 1) * 2 * L::kTileBytes), L::kRegion, 1024);
#pragma unroll
        for (int k = 0; k < 4; ++k)
          mma_ts(tDQ, tDP + (i & 1) * 64 + (k >> 1) * 32 + (k & 1) * 8, k_mn + (uint64_t)(((h * 64 + k * 16) * 128) >> 4), idesc_nn,
                 (i > 0 || k > 0) ? 1u : 0u);
        if (h == 1 || i + 1 == n_steps) mma_commit(&ctrl->walk_free[it & 1]);   // last use of the tile's K and V
        return true;
      };
      mbar_arrive_expect_tx(&ctrl->fix_full, 2 * L::kTileBytes);
      for (int c = 0; c < L::kChunks; ++c) {
        tma_load_3d(smem + L::kFix0 + c * L::kRegion, &tmap_q, &ctrl->fix_full, c * 64, head0, q0);
        tma_load_3d(smem + L::kFix1 + c * L::kRegion, &tmap_do, &ctrl->fix_full, c * 64, head0, q0);
      }
      if (n_iter > 0) load_walk(0);
      if (n_iter > 1) load_walk(1);
      ok = mbar_wait(&ctrl->fix_full, 0, abort_flag);
      int reload = -1;                                   // key tile whose buffer is refilled once its products have completed
      for (int i = 0; i <= n_steps && ok; ++i) {
        if (i < n_steps) ok = issue_scores(i);
        if (ok && reload >= 0) {
          if (reload + 2 < n_iter) {
            ok = mbar_wait(&ctrl->walk_free[reload & 1], (reload >> 1) & 1, abort_flag);
            if (ok) load_walk(reload + 2);
          }
          reload = -1;
        }
        if (ok && i > 0) {
          ok = issue_grads(i - 1);
          if ((i - 1) & 1) reload = (i - 1) >> 1;
        }
      }
      if (ok) mma_commit(&ctrl->fin);
    }
  } else {
    const int r = tid & 127;                             // row of the query tile = tensor-memory lane
    const int ch = tid >> 7;                             // which 32 of a step's 64 columns this thread takes
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const int tok_i = q0 + (r >> p.hpt_log2);
    const int head = head0 + (r & (p.hpt - 1));
    const bool row_ok = tok_i < q_end;
    float lse2 = 0.f, dl = 0.f;
    if (row_ok) {
      lse2 = __ldg(p.lse + (size_t)tok_i * p.Hq + head) * 1.4426950408889634f;
      dl = __ldg(p.delta + (size_t)tok_i * p.Hq + head) * p.scale;
    }
    bool ok = true;
    for (int i = 0; i < n_steps; ++i) {
      const int kr = kv0 + i * 64;
      const int n_ok = row_ok ? max(0, min(64, tok_i - kr + 1)) : 0;
      // every pair of this step visible?  (every row of the tile exists and already the first one sees the step's last key)
      const bool all_visible = q0 + p.tok <= q_end && q0 - kr + 1 >= 64;
      ok = mbar_wait(&ctrl->sd_full[i & 1], (i >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      if (all_visible)
        bwd_row_ds<false>(tS + (i & 1) * 64 + lane_off, tDP + (i & 1) * 64 + lane_off, ch, n_ok, p.scale_log2, lse2, dl, p.scale);
      else
        bwd_row_ds<true>(tS + (i & 1) * 64 + lane_off, tDP + (i & 1) * 64 + lane_off, ch, n_ok, p.scale_log2, lse2, dl, p.scale);
      tc_fence_before();
      mbar_arrive(&ctrl->rows_done[i & 1]);
    }
    if (ok && n_steps > 0) ok = mbar_wait(&ctrl->fin, 0, abort_flag);
    if (ok && n_steps > 0) {
      tc_fence_after();
      store_acc_row<D>(tDQ + lane_off, p.dq, ((size_t)tok_i * p.Hq + head) * D, p.out_f32, row_ok, ch);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && ctrl->abort_flag) ba_record_status(p.status, BA_ERR_TIMEOUT);
  if (warp == kCtlWarp) tmem_dealloc(tmem, 512);
}

// delta[row, head] = dO . O: D / 8 threads per (row, head), each with one 16-byte vector of both operands
template <int D>
__global__ void __launch_bounds__(256)
ba_bwd_delta_kernel(const __nv_bfloat16 *__restrict__ o, const __nv_bfloat16 *__restrict__ d_o, float *__restrict__ delta,
                    int n_rows_heads) {
  constexpr int kLanes = D / 8;                          // 8 or 16 threads per row
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long rh = t / kLanes;
  const int v = (int)(t - rh * kLanes);
  float acc = 0.f;
  if (rh < n_rows_heads) {
    const uint4 a = __ldg(reinterpret_cast<const uint4 *>(o + rh * D) + v);
    const uint4 b = __ldg(reinterpret_cast<const uint4 *>(d_o + rh * D) + v);
    const uint32_t aw[4] = {a.x, a.y, a.z, a.w}, bw[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      acc = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(bw[i] << 16), acc);
      acc = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(bw[i] & 0xffff0000u), acc);
    }
  }
#pragma unroll
  for (int sft = kLanes / 2; sft > 0; sft >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, sft);
  if (rh < n_rows_heads && v == 0) delta[rh] = acc;
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

bool bwd_make_map(CUtensorMap *m, const void *ptr, int D, int heads, long long rows, int box_heads, int box_rows) {
  static EncodeTiledFn enc = nullptr;
  if (!enc) {
    void *fp = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fp, cudaEnableDefault, &q) != cudaSuccess) return false;
    enc = reinterpret_cast<EncodeTiledFn>(fp);
  }
  if (!enc || rows < 1) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)heads * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
ba_status launch_bwd(ba_ctx *ctx, const BwdParams &p, const CUtensorMap &tq, const CUtensorMap &tdo,
                     const CUtensorMap &tk, const CUtensorMap &tv, int n_ktiles_upper, int n_pairs_upper,
                     cudaStream_t stream) {
  const int smem = BwdLayout<D>::kBytes + 1024;
  ba_bwd_dkv_kernel<D><<<dim3((unsigned)n_ktiles_upper, (unsigned)p.Hkv), kBwdThreads, smem, stream>>>(tq, tdo, tk, tv, p);
  BA_CUDA_TRY(cudaGetLastError());
  ba_bwd_dq_kernel<D><<<dim3((unsigned)(2 * n_pairs_upper), (unsigned)(p.Hq / p.hpt)), kBwdThreads, smem, stream>>>(tq, tdo, tk, tv, p);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 2;
  return BA_OK;
}

}  // namespace

// Per-context set-up (device current): the kernels' shared-memory limit is raised once.
ba_status ba_bwd_sm100_setup(ba_ctx *) {
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_bwd_dkv_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdLayout<128>::kBytes + 1024));
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_bwd_dq_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdLayout<128>::kBytes + 1024));
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_bwd_dkv_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdLayout<64>::kBytes + 1024));
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_bwd_dq_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, BwdLayout<64>::kBytes + 1024));
  return BA_OK;
}

ba_status ba_bwd_sm100_launch(ba_ctx *ctx, const void *q, const void *k, const void *v, const void *o,
                              const float *lse, const void *d_o, void *dq, void *dk, void *dv, int out_f32,
                              const ba_segments *seg, int mode, cudaStream_t stream) {
  const int D = ctx->cfg.head_dim, Hq = ctx->cfg.n_q_heads, Hkv = ctx->cfg.n_kv_heads;
  const int T = seg->n_tokens;
  BwdParams p;
  p.lse = lse; p.dq = dq; p.dk = dk; p.dv = dv; p.out_f32 = out_f32; p.status = ctx->dev_status;
  p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
  p.hpt = ba_heads_per_tile(ctx->cfg);
  p.hpt_log2 = p.hpt == 4 ? 2 : p.hpt == 2 ? 1 : 0;
  p.tok = 128 / p.hpt;
  p.scale = ctx->scale;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.mode = mode; p.n_rows = T; p.seg = *seg;
  if (seg->q_tile_tokens != 2 * p.tok || !seg->cu_ktile) return BA_ERR_INVALID_ARG;
  // delta = dO . O sits in the scratch area of the workspace
  const size_t need = (size_t)T * Hq * sizeof(float);
  if (!ctx->workspace || ctx->workspace_bytes < ba_scratch_offset(ctx) + need) return BA_ERR_WORKSPACE;
  float *delta = reinterpret_cast<float *>(reinterpret_cast<char *>(ctx->workspace) + ba_scratch_offset(ctx));
  p.delta = delta;
  const int n_rh = T * Hq;
  const long long threads = (long long)n_rh * (D / 8);
  if (D == 128)
    ba_bwd_delta_kernel<128><<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(
        (const __nv_bfloat16 *)o, (const __nv_bfloat16 *)d_o, delta, n_rh);
  else
    ba_bwd_delta_kernel<64><<<(unsigned)((threads + 255) / 256), 256, 0, stream>>>(
        (const __nv_bfloat16 *)o, (const __nv_bfloat16 *)d_o, delta, n_rh);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 1;
  CUtensorMap tq, tdo, tk, tv;
  if (!bwd_make_map(&tq, q, D, Hq, T, p.hpt, p.tok) || !bwd_make_map(&tdo, d_o, D, Hq, T, p.hpt, p.tok) ||
      !bwd_make_map(&tk, k, D, Hkv, T, 1, kTile) || !bwd_make_map(&tv, v, D, Hkv, T, 1, kTile))
    return BA_ERR_CUDA;
  const int n_ktiles_upper = T / kTile + seg->n_blocks;
  const int n_pairs_upper = seg->n_prompt_items > 0 ? seg->n_prompt_items : T / (2 * p.tok) + seg->n_blocks;
  if (D == 128) return launch_bwd<128>(ctx, p, tq, tdo, tk, tv, n_ktiles_upper, n_pairs_upper, stream);
  return launch_bwd<64>(ctx, p, tq, tdo, tk, tv, n_ktiles_upper, n_pairs_upper, stream);
}

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
//     query tile that sees them (all heads of the group): S and dP by two products, P and dS by its
//     128 row threads (written to shared memory as bf16), then dV += P^T dO and dK += dS^T Q.
//   * ba_bwd_dq_kernel: one CTA owns one query tile (tokens x heads of one KV group, as in the
//     forward kernel) and walks over the key tiles it sees: S, dP, dS as above, dQ += dS K.
// The steps of a tile run one after the other (loads, two products, row work, two products): the
// kernels are simple rather than pipelined.
#include <math.h>

#include "ba_common.cuh"
#include "ba_sm100.cuh"

using namespace sm100;

int ba_heads_per_tile(const ba_config &c);

namespace {

constexpr int kBwdThreads = 160;      // warps 0-3: one thread per tile row (tensor-memory lane); warp 4: loads and MMA issue
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
  static constexpr int kQ = 0, kDO = kTileBytes, kK = 2 * kTileBytes, kV = 3 * kTileBytes;
  static constexpr int kP = 4 * kTileBytes;               // [128 q rows x 128 keys] bf16
  static constexpr int kDS = kP + 2 * kRegion;
  static constexpr int kCtrl = kDS + 2 * kRegion;
  static constexpr int kBytes = kCtrl + 256;
};

struct BwdCtrl {
  uint64_t kv_full, q_full, sd_full, rows_done, acc_done;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ int upper_bound_dev(const int32_t *a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(a + mid) <= x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// One row of P and dS for a 128-key tile: reads the row of S and dP from tensor memory in chunks of 32
// columns, p = exp2(s * scale_log2 - lse_log2) where the mask allows, ds = p (dp - delta) scale, and stores
// both as bf16 in the 128-byte swizzled layout of a [128 rows x 128 keys] tile (two 64-key regions).
// `n_ok`: columns 0 .. n_ok - 1 are visible to this row (0: none).
__device__ __forceinline__ void bwd_row(uint32_t tS, uint32_t tDP, uint8_t *p_s, uint8_t *ds_s, int r, int n_ok,
                                        float scale_log2, float lse_log2, float delta, float scale) {
  const int rb = r * 128, sw = r & 7;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    uint32_t s[32], dp[32];
    tmem_ld_32x32b_x32(tS + c * 32, s);
    tmem_ld_32x32b_x32(tDP + c * 32, dp);
    tmem_wait_ld();
    uint32_t pw[16], dw[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int e0 = c * 32 + 2 * i;
      float p0 = ex2(fmaf(__uint_as_float(s[2 * i]), scale_log2, -lse_log2));
      float p1 = ex2(fmaf(__uint_as_float(s[2 * i + 1]), scale_log2, -lse_log2));
      if (e0 >= n_ok) p0 = 0.f;
      if (e0 + 1 >= n_ok) p1 = 0.f;
      const float d0 = p0 * (__uint_as_float(dp[2 * i]) - delta) * scale;
      const float d1 = p1 * (__uint_as_float(dp[2 * i + 1]) - delta) * scale;
      __nv_bfloat162 pv = __floats2bfloat162_rn(p0, p1), dv = __floats2bfloat162_rn(d0, d1);
      pw[i] = *reinterpret_cast<uint32_t *>(&pv);
      dw[i] = *reinterpret_cast<uint32_t *>(&dv);
    }
    // columns 32 c .. 32 c + 31 = four 16-byte chunks: chunk index 4 c + k of the row
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const int ch = 4 * c + k;
      const int off = (ch >> 3) * (128 * 128) + rb + (((ch & 7) ^ sw) << 4);
      if (p_s) *reinterpret_cast<uint4 *>(p_s + off) = make_uint4(pw[4 * k], pw[4 * k + 1], pw[4 * k + 2], pw[4 * k + 3]);
      *reinterpret_cast<uint4 *>(ds_s + off) = make_uint4(dw[4 * k], dw[4 * k + 1], dw[4 * k + 2], dw[4 * k + 3]);
    }
  }
}

// Writes one accumulator row (D fp32 columns of tensor memory, lane = row) to global memory.
template <int D>
__device__ __forceinline__ void store_acc_row(uint32_t tAcc, void *dst_base, size_t elem_off, int out_f32, bool valid) {
#pragma unroll
  for (int c = 0; c < D / 32; ++c) {
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
  int r1_begin = k0, r1_end = (p.mode == BA_MODE_FULL) ? seq1 : blk1;           // causal range
  int r2_begin = 0, r2_end = 0;                                                 // range that sees all the keys
  if (p.mode == BA_MODE_BLOCK && !is_final) { r2_begin = fin0; r2_end = seq1; }
  const int tiles1 = (r1_end - r1_begin + p.tok - 1) / p.tok, tiles2 = (r2_end - r2_begin + p.tok - 1) / p.tok;
  const int n_chunks = p.G / p.hpt;                                             // head chunks of this KV group
  const int n_iter = (tiles1 + tiles2) * n_chunks;

  if (tid == 0) {
    mbar_init(&ctrl->kv_full, 1); mbar_init(&ctrl->q_full, 1); mbar_init(&ctrl->sd_full, 1);
    mbar_init(&ctrl->rows_done, 128); mbar_init(&ctrl->acc_done, 1);
    ctrl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 4) { tmem_alloc(&ctrl->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctrl->tmem_base;
  volatile int *abort_flag = &ctrl->abort_flag;
  const uint32_t tS = tmem, tDP = tmem + 128, tDV = tmem + 256, tDK = tmem + 384;

  if (warp == 4) {
    if (elect_one()) {
      constexpr uint32_t idesc_nt = make_idesc_bf16(128, kTile, 0);             // both operands K-major
      constexpr uint32_t idesc_tn = make_idesc_bf16(128, D, 1) | (1u << 15);    // both operands MN-major
      const uint64_t q_desc = make_smem_desc(smem_u32(smem + L::kQ), 16, 1024);
      const uint64_t do_desc = make_smem_desc(smem_u32(smem + L::kDO), 16, 1024);
      const uint64_t k_desc = make_smem_desc(smem_u32(smem + L::kK), 16, 1024);
      const uint64_t v_desc = make_smem_desc(smem_u32(smem + L::kV), 16, 1024);
      const uint64_t p_mn = make_smem_desc(smem_u32(smem + L::kP), L::kRegion, 1024);
      const uint64_t ds_mn = make_smem_desc(smem_u32(smem + L::kDS), L::kRegion, 1024);
      const uint64_t do_mn = make_smem_desc(smem_u32(smem + L::kDO), L::kRegion, 1024);
      const uint64_t q_mn = make_smem_desc(smem_u32(smem + L::kQ), L::kRegion, 1024);
      bool ok = true;
      mbar_arrive_expect_tx(&ctrl->kv_full, 2 * L::kTileBytes);
      for (int c = 0; c < L::kChunks; ++c) {
        tma_load_3d(smem + L::kK + c * L::kRegion, &tmap_k, &ctrl->kv_full, c * 64, g, k0);
        tma_load_3d(smem + L::kV + c * L::kRegion, &tmap_v, &ctrl->kv_full, c * 64, g, k0);
      }
      ok = mbar_wait(&ctrl->kv_full, 0, abort_flag);
      for (int it = 0; it < n_iter && ok; ++it) {
        const int ti = it / n_chunks, ch = it - ti * n_chunks;
        const int row0 = ti < tiles1 ? r1_begin + ti * p.tok : r2_begin + (ti - tiles1) * p.tok;
        const int head0 = g * p.G + ch * p.hpt;
        // the products of the previous iteration have read Q, dO, P and dS: the buffers may be refilled
        if (it > 0) { ok = mbar_wait(&ctrl->acc_done, (it - 1) & 1, abort_flag); if (!ok) break; }
        mbar_arrive_expect_tx(&ctrl->q_full, 2 * L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c) {
          tma_load_3d(smem + L::kQ + c * L::kRegion, &tmap_q, &ctrl->q_full, c * 64, head0, row0);
          tma_load_3d(smem + L::kDO + c * L::kRegion, &tmap_do, &ctrl->q_full, c * 64, head0, row0);
        }
        if (it + 1 < n_iter) {                           // the next iteration's tiles are asked into L2 meanwhile
          const int tn = (it + 1) / n_chunks, cn = it + 1 - tn * n_chunks;
          const int rown = tn < tiles1 ? r1_begin + tn * p.tok : r2_begin + (tn - tiles1) * p.tok;
          for (int c = 0; c < L::kChunks; ++c) {
            tma_prefetch_3d(&tmap_q, c * 64, g * p.G + cn * p.hpt, rown);
            tma_prefetch_3d(&tmap_do, c * 64, g * p.G + cn * p.hpt, rown);
          }
        }
        ok = mbar_wait(&ctrl->q_full, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tS, q_desc + off, k_desc + off, idesc_nt, k > 0);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tDP, do_desc + off, v_desc + off, idesc_nt, k > 0);
        }
        mma_commit(&ctrl->sd_full);
        // the row threads turn S and dP into P and dS in shared memory
        ok = mbar_wait(&ctrl->rows_done, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < kTile / 16; ++k) {           // contraction over the 128 query rows, 16 at a time
          const uint64_t off = (uint64_t)((k * 2048) >> 4);
          mma_ss(tDV, p_mn + off, do_mn + off, idesc_tn, (it > 0 || k > 0) ? 1u : 0u);
        }
#pragma unroll
        for (int k = 0; k < kTile / 16; ++k) {
          const uint64_t off = (uint64_t)((k * 2048) >> 4);
          mma_ss(tDK, ds_mn + off, q_mn + off, idesc_tn, (it > 0 || k > 0) ? 1u : 0u);
        }
        mma_commit(&ctrl->acc_done);
      }
    }
  } else {
    const int r = tid;                                   // row of the query tile = tensor-memory lane
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int ti = it / n_chunks, ch = it - ti * n_chunks;
      const bool causal = ti < tiles1;
      const int row0 = causal ? r1_begin + ti * p.tok : r2_begin + (ti - tiles1) * p.tok;
      const int row_end = causal ? r1_end : r2_end;
      const int tok_i = row0 + (r >> p.hpt_log2);
      const int head = g * p.G + ch * p.hpt + (r & (p.hpt - 1));
      const bool row_ok = tok_i < row_end;
      int n_ok = 0;                                      // visible key columns of this row
      if (row_ok) n_ok = causal ? min(n_keys, tok_i - k0 + 1) : n_keys;
      float lse2 = 0.f, dl = 0.f;
      if (row_ok) {
        lse2 = __ldg(p.lse + (size_t)tok_i * p.Hq + head) * 1.4426950408889634f;
        dl = __ldg(p.delta + (size_t)tok_i * p.Hq + head);
      }
      ok = mbar_wait(&ctrl->sd_full, it & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      bwd_row(tS + lane_off, tDP + lane_off, smem + L::kP, smem + L::kDS, r, n_ok, p.scale_log2, lse2, dl, p.scale);
      tc_fence_before();
      fence_proxy_async();                               // the tensor core reads P and dS through the async proxy
      mbar_arrive(&ctrl->rows_done);
    }
    // accumulators: lane = key row of the tile
    if (ok && n_iter > 0) ok = mbar_wait(&ctrl->acc_done, (n_iter - 1) & 1, abort_flag);
    if (ok) {
      tc_fence_after();
      const bool valid = r < n_keys;
      const size_t off = ((size_t)(k0 + r) * p.Hkv + g) * D;
      if (n_iter > 0) {
        store_acc_row<D>(tDV + lane_off, p.dv, off, p.out_f32, valid);
        store_acc_row<D>(tDK + lane_off, p.dk, off, p.out_f32, valid);
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && ctrl->abort_flag) ba_record_status(p.status, BA_ERR_TIMEOUT);
  if (warp == 4) tmem_dealloc(tmem, 512);
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

  if (tid == 0) {
    mbar_init(&ctrl->kv_full, 1); mbar_init(&ctrl->q_full, 1); mbar_init(&ctrl->sd_full, 1);
    mbar_init(&ctrl->rows_done, 128); mbar_init(&ctrl->acc_done, 1);
    ctrl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 4) { tmem_alloc(&ctrl->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctrl->tmem_base;
  volatile int *abort_flag = &ctrl->abort_flag;
  const uint32_t tS = tmem, tDP = tmem + 128, tDQ = tmem + 256;

  if (warp == 4) {
    if (elect_one()) {
      constexpr uint32_t idesc_nt = make_idesc_bf16(128, kTile, 0);
      constexpr uint32_t idesc_nn = make_idesc_bf16(128, D, 1);                 // A K-major (dS), B MN-major (K)
      const uint64_t q_desc = make_smem_desc(smem_u32(smem + L::kQ), 16, 1024);
      const uint64_t do_desc = make_smem_desc(smem_u32(smem + L::kDO), 16, 1024);
      const uint64_t k_desc = make_smem_desc(smem_u32(smem + L::kK), 16, 1024);
      const uint64_t v_desc = make_smem_desc(smem_u32(smem + L::kV), 16, 1024);
      const uint64_t ds_desc = make_smem_desc(smem_u32(smem + L::kDS), 16, 1024);
      const uint64_t k_mn = make_smem_desc(smem_u32(smem + L::kK), L::kRegion, 1024);
      bool ok = true;
      mbar_arrive_expect_tx(&ctrl->q_full, 2 * L::kTileBytes);
      for (int c = 0; c < L::kChunks; ++c) {
        tma_load_3d(smem + L::kQ + c * L::kRegion, &tmap_q, &ctrl->q_full, c * 64, head0, q0);
        tma_load_3d(smem + L::kDO + c * L::kRegion, &tmap_do, &ctrl->q_full, c * 64, head0, q0);
      }
      ok = mbar_wait(&ctrl->q_full, 0, abort_flag);
      for (int it = 0; it < n_iter && ok; ++it) {
        const int kr = kv0 + it * kTile;
        if (it > 0) { ok = mbar_wait(&ctrl->acc_done, (it - 1) & 1, abort_flag); if (!ok) break; }   // K, V, dS free again
        mbar_arrive_expect_tx(&ctrl->kv_full, 2 * L::kTileBytes);
        for (int c = 0; c < L::kChunks; ++c) {
          tma_load_3d(smem + L::kK + c * L::kRegion, &tmap_k, &ctrl->kv_full, c * 64, g, kr);
          tma_load_3d(smem + L::kV + c * L::kRegion, &tmap_v, &ctrl->kv_full, c * 64, g, kr);
        }
        if (it + 1 < n_iter)
          for (int c = 0; c < L::kChunks; ++c) {
            tma_prefetch_3d(&tmap_k, c * 64, g, kr + kTile);
            tma_prefetch_3d(&tmap_v, c * 64, g, kr + kTile);
          }
        ok = mbar_wait(&ctrl->kv_full, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tS, q_desc + off, k_desc + off, idesc_nt, k > 0);
        }
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          mma_ss(tDP, do_desc + off, v_desc + off, idesc_nt, k > 0);
        }
        mma_commit(&ctrl->sd_full);
        ok = mbar_wait(&ctrl->rows_done, it & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int k = 0; k < kTile / 16; ++k) {           // contraction over the 128 keys of the tile
          const uint64_t a_off = (uint64_t)(((k >> 2) * L::kRegion + (k & 3) * 32) >> 4);
          const uint64_t b_off = (uint64_t)((k * 2048) >> 4);
          mma_ss(tDQ, ds_desc + a_off, k_mn + b_off, idesc_nn, (it > 0 || k > 0) ? 1u : 0u);
        }
        mma_commit(&ctrl->acc_done);
      }
    }
  } else {
    const int r = tid;
    const uint32_t lane_off = (uint32_t)(warp * 32) << 16;
    const int tok_i = q0 + (r >> p.hpt_log2);
    const int head = head0 + (r & (p.hpt - 1));
    const bool row_ok = tok_i < q_end;
    float lse2 = 0.f, dl = 0.f;
    if (row_ok) {
      lse2 = __ldg(p.lse + (size_t)tok_i * p.Hq + head) * 1.4426950408889634f;
      dl = __ldg(p.delta + (size_t)tok_i * p.Hq + head);
    }
    bool ok = true;
    for (int it = 0; it < n_iter; ++it) {
      const int kr = kv0 + it * kTile;
      const int n_ok = row_ok ? max(0, min(kTile, tok_i - kr + 1)) : 0;
      ok = mbar_wait(&ctrl->sd_full, it & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      bwd_row(tS + lane_off, tDP + lane_off, nullptr, smem + L::kDS, r, n_ok, p.scale_log2, lse2, dl, p.scale);
      tc_fence_before();
      fence_proxy_async();
      mbar_arrive(&ctrl->rows_done);
    }
    if (ok && n_iter > 0) ok = mbar_wait(&ctrl->acc_done, (n_iter - 1) & 1, abort_flag);
    if (ok && n_iter > 0) {
      tc_fence_after();
      store_acc_row<D>(tDQ + lane_off, p.dq, ((size_t)tok_i * p.Hq + head) * D, p.out_f32, row_ok);
    }
  }
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && ctrl->abort_flag) ba_record_status(p.status, BA_ERR_TIMEOUT);
  if (warp == 4) tmem_dealloc(tmem, 512);
}

// delta[row, head] = dO . O
template <int D>
__global__ void __launch_bounds__(256)
ba_bwd_delta_kernel(const __nv_bfloat16 *__restrict__ o, const __nv_bfloat16 *__restrict__ d_o, float *__restrict__ delta,
                    int n_rows_heads) {
  const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (warp >= n_rows_heads) return;
  const __nv_bfloat162 *a = reinterpret_cast<const __nv_bfloat162 *>(o + (size_t)warp * D);
  const __nv_bfloat162 *b = reinterpret_cast<const __nv_bfloat162 *>(d_o + (size_t)warp * D);
  float acc = 0.f;
  for (int i = lane; i < D / 2; i += 32) {
    const float2 x = __bfloat1622float2(a[i]), y = __bfloat1622float2(b[i]);
    acc = fmaf(x.x, y.x, acc);
    acc = fmaf(x.y, y.y, acc);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) delta[warp] = acc;
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
  const long long threads = (long long)n_rh * 32;
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

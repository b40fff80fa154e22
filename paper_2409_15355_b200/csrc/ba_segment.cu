// Segment tables of a ragged batch (Section 2.2: one passage per block, the user
// query is the final block; Section 2.5: a block's positions follow from its
// place in the prompt; Section 2.3: cached blocks start at position zero, so the
// re-encoding delta of a block is the prompt position of its first token).
//
// Two kernels.  The first runs as one CTA and turns the length arrays into
// prefix sums with warp-shuffle scans (the arrays are a few hundred entries, a
// single CTA keeps every scan's carry in registers).  The second resolves the
// per-token tables with one binary search per token.
#include "ba_common.cuh"

namespace {

constexpr int kScanThreads = 1024;

// CTA-wide exclusive scan of one int per thread.  Returns the exclusive prefix of
// `v` and sets `total` to the sum over the CTA.  `smem` holds 33 ints.
__device__ __forceinline__ int cta_exclusive_scan(int v, int *smem, int &total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int n = __shfl_up_sync(0xffffffffu, inc, d);
    if (lane >= d) inc += n;
  }
  __syncthreads();  // smem reuse across consecutive scans
  if (lane == 31) smem[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    int w = smem[lane];
    int winc = w;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      int n = __shfl_up_sync(0xffffffffu, winc, d);
      if (lane >= d) winc += n;
    }
    smem[lane] = winc - w;  // exclusive prefix of the warp totals
    if (lane == 31) smem[32] = winc;
  }
  __syncthreads();
  total = smem[32];
  return smem[warp] + inc - v;
}

// First index in a[0..n) whose value is > x (a ascending).
__device__ __forceinline__ int upper_bound(const int32_t *a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (a[mid] <= x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

__global__ void __launch_bounds__(kScanThreads)
ba_segment_blocks_kernel(const int32_t *__restrict__ lens, const int32_t *__restrict__ seq_nblocks,
                         int batch, int B, int T, int mode, int tile_tok, int gen, ba_segments seg,
                         int32_t *status) {
  __shared__ int scan_smem[33];
  __shared__ int bad;
  const int tid = threadIdx.x;
  if (tid == 0) { bad = 0; seg.totals[7] = 0; seg.totals[6] = gen; }   // [6]: stamp of this call
  __syncthreads();

  // --- first block of every sequence
  int carry = 0;
  for (int base = 0; base < batch; base += kScanThreads) {
    int s = base + tid;
    int nb = (s < batch) ? seq_nblocks[s] : 0;
    if (s < batch && nb < 1) { bad = 1; nb = 0; }
    int total;
    int ex = cta_exclusive_scan(nb, scan_smem, total);
    if (s < batch) seg.cu_seq_block[s] = carry + ex;
    carry += total;
  }
  if (tid == 0) seg.cu_seq_block[batch] = carry;
  __syncthreads();
  if (carry != B || bad) {  // uniform: every thread holds the same carry and reads the same flag
    if (tid == 0) ba_record_status(status, BA_ERR_INVALID_ARG);
    return;
  }

  // --- per-block prefix sums: rows (prompt, cache, final packing) and query tiles
  int c_all = 0, c_cache = 0, c_final = 0, c_tile = 0, c_ktile = 0, c_atile = 0;
  for (int base = 0; base < B; base += kScanThreads) {
    int b = base + tid;
    int len = 0, fin = 0, s = 0;
    if (b < B) {
      len = lens[b];
      if (len < 1) { bad = 1; len = 0; }
      s = upper_bound(seg.cu_seq_block, batch + 1, b) - 1;
      fin = (b == seg.cu_seq_block[s + 1] - 1);
    }
    int t_all, t_cache, t_final, t_tile, t_ktile;
    int e_all = cta_exclusive_scan(len, scan_smem, t_all);
    int e_cache = cta_exclusive_scan(fin ? 0 : len, scan_smem, t_cache);
    int e_final = cta_exclusive_scan(fin ? len : 0, scan_smem, t_final);
    int e_tile = cta_exclusive_scan((len + tile_tok - 1) / tile_tok, scan_smem, t_tile);
    int e_ktile = cta_exclusive_scan(fin ? 0 : (len + 127) / 128, scan_smem, t_ktile);
    int t_atile;
    int e_atile = cta_exclusive_scan((len + 127) / 128, scan_smem, t_atile);
    if (b < B) {
      seg.cu_block[b] = c_all + e_all;
      seg.block_seq[b] = s;
      seg.block_is_final[b] = (uint8_t)fin;
      seg.block_part_off[b] = fin ? (c_final + e_final) : (c_cache + e_cache);
      seg.cu_qtile[b] = c_tile + e_tile;
      seg.cu_ktile[b] = c_atile + e_atile;
      if (!fin) {
        // every earlier sequence contributed exactly one final block
        int c = b - s;
        seg.cache_block[c] = b;
        seg.cache_cu[c] = c_cache + e_cache;
        seg.cache_tile_cu[c] = c_ktile + e_ktile;
      }
    }
    c_all += t_all; c_cache += t_cache; c_final += t_final; c_tile += t_tile; c_ktile += t_ktile; c_atile += t_atile;
  }
  if (tid == 0) {
    seg.cu_block[B] = c_all;
    seg.cache_cu[B - batch] = c_cache;
    seg.cache_tile_cu[B - batch] = c_ktile;
    seg.cu_qtile[B] = c_tile;
    seg.cu_ktile[B] = c_atile;
    seg.totals[0] = c_cache;
    seg.totals[1] = c_final;
    seg.totals[2] = c_tile;
    if (c_all != T) bad = 1;
  }
  __syncthreads();

  // --- deltas and visibility ranges
  for (int b = tid; b < B; b += kScanThreads) {
    int s = seg.block_seq[b];
    int seq_start = seg.cu_block[seg.cu_seq_block[s]];
    int start = seg.cu_block[b];
    int fin = seg.block_is_final[b];
    seg.block_delta[b] = start - seq_start;
    seg.block_kv_begin[b] = (mode == BA_MODE_FULL || fin) ? seq_start : start;
    if (!fin) seg.cache_delta[b - s] = start - seq_start;
  }

  // --- per-sequence offsets in the three packings, final-block tiles
  int f_rows = 0, f_tiles = 0;
  for (int base = 0; base < batch; base += kScanThreads) {
    int s = base + tid;
    int flen = 0;
    if (s < batch) {
      flen = lens[seg.cu_seq_block[s + 1] - 1];
      if (flen < 1) flen = 0;
    }
    int t_rows, t_tiles;
    int e_rows = cta_exclusive_scan(flen, scan_smem, t_rows);
    int e_tiles = cta_exclusive_scan((flen + tile_tok - 1) / tile_tok, scan_smem, t_tiles);
    if (s < batch) {
      int start = seg.cu_block[seg.cu_seq_block[s]];
      seg.cu_seq[s] = start;
      seg.cu_final_seq[s] = f_rows + e_rows;
      seg.cu_cache_seq[s] = start - (f_rows + e_rows);
      seg.cu_ftile[s] = f_tiles + e_tiles;
    }
    f_rows += t_rows; f_tiles += t_tiles;
  }
  if (tid == 0) {
    seg.cu_seq[batch] = c_all;
    seg.cu_final_seq[batch] = f_rows;
    seg.cu_cache_seq[batch] = c_all - f_rows;
    seg.cu_ftile[batch] = f_tiles;
    seg.totals[3] = f_tiles;
  }
  __syncthreads();
  if (tid == 0) {
    if (bad) ba_record_status(status, BA_ERR_INVALID_ARG);
    else seg.totals[7] = BA_TABLES_VALID;  // kernels that walk the tables check this word first
  }
}

__global__ void __launch_bounds__(256)
ba_segment_tokens_kernel(int B, int T, ba_segments seg) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= T) return;
  if (seg.totals[7] != BA_TABLES_VALID) return;
  int b = upper_bound(seg.cu_block, B + 1, i) - 1;
  b = min(max(b, 0), B - 1);
  int local = i - seg.cu_block[b];
  seg.tok_block[i] = b;
  seg.tok_pos_local[i] = local;
  seg.tok_pos[i] = seg.block_delta[b] + local;
}

}  // namespace

ba_status ba_segment_launch(ba_ctx *ctx, const int32_t *d_block_lens, const int32_t *d_seq_nblocks,
                            int32_t batch, int32_t n_blocks, int32_t n_tokens, int mode, int32_t gen,
                            const ba_segments *seg, cudaStream_t stream) {
  ba_segment_blocks_kernel<<<1, kScanThreads, 0, stream>>>(
      d_block_lens, d_seq_nblocks, batch, n_blocks, n_tokens, mode, seg->q_tile_tokens, gen, *seg,
      ctx->dev_status);
  BA_CUDA_TRY(cudaGetLastError());
  ba_segment_tokens_kernel<<<(n_tokens + 255) / 256, 256, 0, stream>>>(n_blocks, n_tokens, *seg);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 2;
  return BA_OK;
}

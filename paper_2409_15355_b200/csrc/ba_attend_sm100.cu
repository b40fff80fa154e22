// Tensor-core attention under the Block-attention mask for sm_100a.
//
// One kernel serves ba_block_prefill (Section 1 / 2.4: a row of a non-final block
// sees its own block, causally; a row of a final block sees its whole sequence
// prefix) and ba_final_attend (Section 2.5 step 3: the final block over the
// re-encoded cached blocks plus itself).  The mask never exists as a matrix: a
// work item is a pair of query tiles of one block, its keys are one optional
// "cached" range (all visible) followed by one "own" range (causal).
//
// Structure of a CTA (384 threads, one CTA per SM):
//   warps 0-3   softmax of query tile 0      (one thread per tile row = TMEM lane)
//   warps 4-7   softmax of query tile 1
//   warp  8     TMA producer: Q tiles once, then K_j, V_j, K_j+1, ... into a ring of stages
//   warp  9     MMA issuer (one elected thread): S = Q K^T and O += P V with tcgen05.mma,
//               accumulators in tensor memory (S0, S1, O0, O1 = 4 x 128 columns)
// A query tile is 128 rows = (128 / HPT) tokens x HPT query heads of one KV group,
// so a K/V tile staged once serves every head of the group and both query tiles.
// Softmax is online in fp32 (base-2 exponent with the scale folded in); P is
// written back to tensor memory as bf16 over the S columns and used as the A
// operand of the PV product.  O is rescaled in tensor memory only when the
// running maximum grows by more than 2^8, which keeps every term bounded and the
// result exact in real arithmetic.
//
// Fused warm path (Section 2.5 steps 2 and 3 in one launch): the cached keys stay at their
// cache-time positions and the position difference of each block (Eq. 3 after Eq. 2) is applied
// to the other side of the dot product, (R(p) q) . (R(delta + t) k) = (R(-delta) R(p) q) . (R(t) k):
// each softmax thread owns one row of its query tile and prepares, for every cached block of the
// work entry, a copy of that row rotated by the block's delta (and a plain copy for the final
// block's own keys) in one of two buffers per query tile.  The copy for the next block is made
// while the current block's tiles are worked on -- the plain tile is fetched after one tile and
// rotated in place after the next, in time the thread would otherwise spend waiting for S --
// so the QK^T products switch buffers without a pause.  The cached keys are never rewritten or
// re-read, and a key tile never spans two blocks.
#include <math.h>
#include <new>
#include <type_traits>

#include "ba_common.cuh"
#include "ba_sm100.cuh"
#include "ba_reencode_dev.cuh"

using namespace sm100;

// Tuning aid, absent from ordinary builds: with -DBA_TRACE the roles of CTA 0 stamp clock64() at the
// phases of their first 64 key tiles into a device array that a developer build reads back
// (roles 0/1: softmax groups, 2: MMA thread per query tile, 3: MMA thread's K/V waits, 5: fused query versions).
#ifdef BA_TRACE
__device__ long long g_ba_trace[6][64][8];
extern "C" int ba_trace_read(long long *dst) { return (int)cudaMemcpyFromSymbol(dst, g_ba_trace, sizeof(g_ba_trace)); }
#define BA_TR(role, tile, k)                                                                  \
  do {                                                                                        \
    if (blockIdx.x == 0 && (tile) < 64) g_ba_trace[role][tile][k] = clock64(); \
  } while (0)
#else
#define BA_TR(role, tile, k) do { } while (0)
#endif

namespace {

constexpr int kThreads = 384;
constexpr int kBlockN = 128;      // keys per tile
constexpr int kStages = 3;           // ring of K/V tiles (K_j, V_j, K_j+1, ...)
constexpr float kRescaleThreshold = 8.0f;
constexpr int kBgStageBytes = 16384; // two spare warps x two stages of source rows
constexpr int kWorkSlots = 4;      // ring of published work entries (power of two)
constexpr int kBalTableOff = 512;  // balanced launch: prefix table of front tiles, in the control area behind Ctrl
// (its capacity, kBalMaxPairs items per head chunk, is declared with the planning arithmetic; the spare warps' barriers follow at 1024)
// Register split after launch (168 per thread): the service warps give registers to the softmax warps.
// 128 * kServiceRegs + 256 * kSoftmaxRegs <= 384 * 168.  The MMA thread keeps a work entry, descriptors
// and ring positions live and spills below about 88; the softmax warps start to spill below 208.  On the
// fused path the softmax warps also prepare query versions and need the larger share.
constexpr int kServiceRegsPlain = 88, kSoftmaxRegsPlain = 208;
constexpr int kServiceRegsFused = 72, kSoftmaxRegsFused = 216;

struct AttnParams {
  void *o;
  float *lse;
  int32_t *status;
  int out_f32;
  int Hq, Hkv, G;
  int hpt, hpt_log2, tok;         // heads per tile, tokens per tile (hpt * tok = 128)
  float scale, scale_log2;
  int final_only;
  int n_q_rows;
  int n_chunks;                   // head chunks per token (Hq / hpt)
  int n_splits;                   // > 1: the key tiles of an item are divided among n_splits work entries, combined later
  float *o_part;                  // [n_splits, n_q_rows, Hq, D] fp32, each normalised by its own denominator
  float *lse_part;                // [n_splits, n_q_rows, Hq] natural-log denominators (-inf: split saw no key)
  const int32_t *v_src_off;       // non-null: values of cached block c start at pool row v_src_off[c]
  int persistent;                 // 1: CTAs draw work from counters[0]; 0: CTA b handles entry b only
  // balanced > 0 (final block over a long cache, fewer items than CTAs): the first `balanced` CTAs each take the
  // last bal_len key tiles of one item (slot 0 of its partial results); the other CTAs share the key tiles in
  // front of those, cut into equal runs whatever item they fall in (slots 1 ..).  n_splits is the slot count.
  int balanced, bal_len;
  int q_double;                   // plain path, no background job: two pairs of query buffers (see Ctrl)
  // three device words, zero at launch and zero again when the launch ends (its last CTA clears them):
  // [0] next entry of the work list, [1] next chunk of the background job, [2] CTAs that have finished
  int32_t *counters;
  ba_reencode_job bg;             // bg.n_rows > 0: a re-encoding job the two spare warps carry out meanwhile
  int bg_rows_per_chunk;
  ba_segments seg;
  const int32_t *k_src_off;       // non-null: keys of cached block c start at pool row k_src_off[c] (fused path only)
  int walk;                       // cached keys are walked block by block (a tile never spans two blocks)
  // paged pool: cached block c owns the pages page_idx[page_cu[c] .. page_cu[c+1]) of 1 << page_lg rows each;
  // row t of the block is row t & (page_rows - 1) of page t >> page_lg of its list.  Applies to the values
  // (v_paged) and, on the fused path, to the keys (k_paged).
  const int32_t *page_cu, *page_idx;
  int page_lg, k_paged, v_paged;
  int fused;                      // cached keys are at cache-time positions: queries are counter-rotated per block
  int rope_layout;
  const float2 *q_rope;           // fused: [cached blocks][D/2] (cos, sin) of delta_c * theta_m
};

template <int D>
struct Layout {
  static constexpr int kChunks = D / 64;                  // 64-column (128-byte) swizzle regions per row
  static constexpr int kTileBytes = 128 * D * 2;          // one 128-row tile of Q, K or V
  static constexpr int kRegionBytes = 128 * 128;          // 128 rows x 128 bytes
  static constexpr int kQ0 = 0;
  static constexpr int kQ1 = kTileBytes;
  static constexpr int kRing = 2 * kTileBytes;
  static constexpr int kCtrl = kRing + kStages * kTileBytes;   // 2 KB: Ctrl, then two ba_bg_smem
  static constexpr int kBg = kCtrl + 2048;                     // staging of the background re-encoding, or (fused
                                                               // path) the second pair of query tile buffers
  static constexpr int kBytes = kBg + 4 * kBgStageBytes;
};

// What the scheduling thread publishes to the other roles of its CTA.
struct WorkEntry {
  int pair;            // item (index into the list of query tile pairs); < 0: no more work
  int unit;            // the sequence (final attend) or block (prefill) of the item
  int chunk;           // head chunk
  int tile0, n_tiles;  // key tiles [tile0, tile0 + n_tiles) of the item
  int split;           // slot of the partial results this entry writes
  int fill;            // slots fill .. n_splits - 1 of the item stay unused: this entry marks them empty
};

struct Ctrl {
  // [buffer pair][query tile].  Plain path without a background job: the query tiles of successive entries
  // alternate between two pairs of buffers, so the next entry's queries are fetched while the current one runs.
  uint64_t q_full[2][2];
  uint64_t q_empty[2];            // every QK^T of the entry that used this buffer pair has completed: it may be reloaded
  uint64_t kv_full[kStages];
  uint64_t kv_empty[kStages];
  uint64_t s_full[2];
  uint64_t p_full[2][2];          // [query tile][half of the P tile]
  uint64_t o_done[2];
  uint64_t o_free[2];             // the softmax warps have read O_t out of tensor memory
  uint64_t work_full[kWorkSlots];  // work entry published by the scheduler (producer thread)
  uint64_t work_empty[kWorkSlots]; // entry read by the MMA thread and the 8 softmax warps
  WorkEntry work_ring[kWorkSlots];
  int tile_valid[8];              // pool mode: valid key columns of the cached tiles in flight
  uint32_t tmem_base;
  int abort_flag;
  uint64_t qr_full[2][2];         // fused: [query tile][buffer] the tile prepared for the next key range is ready
  uint64_t cs_full[2];            // fused: the block's (cos, sin) row has been staged for softmax group t
  uint64_t qraw_full[2];          // fused: the plain query tile t has landed in the buffer of the version being prepared
};
static_assert(sizeof(Ctrl) <= kBalTableOff && kBalTableOff + (kBalMaxPairs + 1) * 4 <= 1024, "control area layout");

// One work item: two query tiles of one block (or final block) and the key ranges they see.
struct Item {
  int q_row0;        // first query row (q packing)
  int q_rows;        // valid query rows in the pair (1 .. 2*tok)
  int n_qt;          // 1 or 2 query tiles in use
  int cache_row0, cache_len;   // cached keys (cache packing), all visible
  int own_row0;      // first own key row (q packing); row i sees own rows own_row0 .. i
  int n_cache_tiles, n_tiles;
  int cb0;           // index (cache order) of the sequence's first cached block
  int ctile0;        // cache_tile_cu[cb0]: pool mode walks cached keys block by block
};

__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}

__device__ __forceinline__ int upper_bound_tbl(const int32_t *a, int n, int x) {
  int lo = 0, hi = n;
  while (lo < hi) {
    int mid = (lo + hi) >> 1;
    if (__ldg(a + mid) <= x) lo = mid + 1; else hi = mid;
  }
  return lo;
}

// The sequence (final attend) or block (prefill) that item `pair` belongs to; -1 past the end of the list.
__device__ __forceinline__ int find_unit(const AttnParams &p, int pair) {
  const ba_segments &sg = p.seg;
  if (p.final_only) {
    if (pair >= __ldg(sg.totals + 3)) return -1;
    if (sg.batch == 1) return 0;
    return upper_bound_tbl(sg.cu_ftile, sg.batch + 1, pair) - 1;
  }
  if (pair >= __ldg(sg.totals + 2)) return -1;
  return upper_bound_tbl(sg.cu_qtile, sg.n_blocks + 1, pair) - 1;
}

// Item `pair` of sequence / block `unit`.  The table look-ups are independent of one another (the search for the
// unit, a chain of dependent loads, is done once by the scheduling thread and published with the entry).
__device__ __forceinline__ bool resolve_item(const AttnParams &p, int pair, int unit, Item &it) {
  const ba_segments &sg = p.seg;
  const int pair_tok = 2 * p.tok;
  if (unit < 0) return false;
  if (p.final_only) {
    const int s = unit;
    int f0 = __ldg(sg.cu_final_seq + s), f1 = __ldg(sg.cu_final_seq + s + 1);
    it.q_row0 = f0 + (pair - __ldg(sg.cu_ftile + s)) * pair_tok;
    it.q_rows = min(pair_tok, f1 - it.q_row0);
    it.cache_row0 = __ldg(sg.cu_cache_seq + s);
    it.cache_len = __ldg(sg.cu_cache_seq + s + 1) - it.cache_row0;
    it.own_row0 = f0;
    it.cb0 = __ldg(sg.cu_seq_block + s) - s;           // every earlier sequence has one final block
    it.ctile0 = p.walk ? __ldg(sg.cache_tile_cu + it.cb0) : 0;
    it.n_cache_tiles = p.walk ? __ldg(sg.cache_tile_cu + (__ldg(sg.cu_seq_block + s + 1) - s - 1)) - it.ctile0
                                   : (it.cache_len + kBlockN - 1) / kBlockN;
  } else {
    const int b = unit;
    int b0 = __ldg(sg.cu_block + b), b1 = __ldg(sg.cu_block + b + 1);
    it.q_row0 = b0 + (pair - __ldg(sg.cu_qtile + b)) * pair_tok;
    it.q_rows = min(pair_tok, b1 - it.q_row0);
    it.cache_row0 = 0;
    it.cache_len = 0;
    it.own_row0 = __ldg(sg.block_kv_begin + b);
    it.cb0 = 0; it.ctile0 = 0; it.n_cache_tiles = 0;
  }
  if (it.q_rows < 1) return false;
  it.n_qt = it.q_rows > p.tok ? 2 : 1;
  it.n_tiles = it.n_cache_tiles + (it.q_row0 + it.q_rows - it.own_row0 + kBlockN - 1) / kBlockN;
  return true;
}

// One entry of a CTA's work list: an item, the heads it covers and its share of the key tiles.
struct Work {
  Item it;
  int head0, kv_head;
  int tile0, n_tiles;   // key tiles [tile0, tile0 + n_tiles) of the item (split-KV share)
  int split, fill;
};

// Entry w of the global work list (equal shares of every item's key tiles).  pair < 0 past the end.
//  Prefill: items heaviest-first (descending pair index: within a sequence an item's cost grows
//  with its index, the final block comes last), then head chunk, then split.
//  Final attend: all items cost about the same, so the pair index varies fastest instead: the
//  CTAs running at the same time then work on the same (KV head, key range) for different query
//  tiles and each K/V tile comes from HBM once and from L2 for the others.
__device__ __forceinline__ WorkEntry list_entry(const AttnParams &p, int w) {
  WorkEntry e = {-1, -1, 0, 0, 0, 0, 0};
  const int per_pair = p.n_chunks * p.n_splits;
  const int total_pairs = __ldg(p.seg.totals + (p.final_only ? 3 : 2));
  int rank, rem;
  if (p.final_only) {
    if (total_pairs <= 0) return e;
    rem = w / total_pairs; rank = w - rem * total_pairs;
    if (rem >= per_pair) return e;
  } else {
    rank = w / per_pair; rem = w - rank * per_pair;
    if (rank >= total_pairs) return e;
  }
  Item it;
  e.unit = find_unit(p, total_pairs - 1 - rank);
  if (!resolve_item(p, total_pairs - 1 - rank, e.unit, it)) return e;
  e.pair = total_pairs - 1 - rank;
  e.chunk = rem / p.n_splits;
  e.split = rem - e.chunk * p.n_splits;
  e.fill = p.n_splits;
  e.tile0 = (int)(((long long)it.n_tiles * e.split) / p.n_splits);
  e.n_tiles = (int)(((long long)it.n_tiles * (e.split + 1)) / p.n_splits) - e.tile0;
  return e;
}

// A published entry, decoded by the role that reads it.  Returns false at the end of the work.
__device__ __forceinline__ bool load_work(const AttnParams &p, const WorkEntry &e, Work &wk) {
  if (e.pair < 0 || !resolve_item(p, e.pair, e.unit, wk.it)) return false;
  wk.head0 = e.chunk * p.hpt;
  wk.kv_head = wk.head0 / p.G;
  wk.tile0 = e.tile0;
  wk.n_tiles = e.n_tiles;
  wk.split = e.split;
  wk.fill = e.fill;
  return true;
}

// The last own key tile of an item covers the diagonal of the causal range.  When every row of the item
// ends in the tile's first 64 keys (true for every other item: items are 64-token aligned, key tiles 128),
// its second half is masked for all of them: the products and the exponentials of that half are skipped.
__device__ __forceinline__ bool last_tile_is_half(const Work &wk) {
  const Item &it = wk.it;
  if (wk.tile0 + wk.n_tiles != it.n_tiles || it.n_tiles == it.n_cache_tiles) return false;   // the entry does not end the item
  const int last_key0 = it.own_row0 + (it.n_tiles - it.n_cache_tiles - 1) * kBlockN;
  return it.q_row0 + it.q_rows - 1 - last_key0 < kBlockN / 2;
}

// Block-by-block walk of the cached keys: index (cache order) of the block that holds key tile
// `target` (counted over the whole batch); the sequence's blocks follow cb0.
__device__ __forceinline__ int find_cache_block(const AttnParams &p, const Item &it, int target) {
  int lo = it.cb0, hi = p.seg.n_cached_blocks;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (__ldg(p.seg.cache_tile_cu + mid) <= target) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Counter-rotation of query rows [row_begin, row_end) of one tile (fused warm path): dst = R(-delta) src,
// with cs = (cos, sin)(delta * theta_m) of the current cached block.  Both tiles are in the 128-byte
// swizzled layout the tensor maps produce: 64-column regions of 128 rows x 128 bytes, the 16-byte
// chunk c of row r stored at chunk position c ^ (r & 7).  Called by one full warp; a lane keeps its
// chunk column, so its (cos, sin) values are loaded once per block.
__device__ __forceinline__ uint32_t rot_word_adjacent(uint32_t w, float2 cs) {
  const float x = __uint_as_float(w << 16), y = __uint_as_float(w & 0xffff0000u);
  __nv_bfloat162 v = __floats2bfloat162_rn(fmaf(x, cs.x, y * cs.y), fmaf(y, cs.x, -x * cs.y));
  return *reinterpret_cast<uint32_t *>(&v);
}
__device__ __forceinline__ void rot_words_half(uint32_t &a, uint32_t &b, float2 cs0, float2 cs1) {
  // a holds x of pairs m, m+1; b holds their partners y
  const float x0 = __uint_as_float(a << 16), x1 = __uint_as_float(a & 0xffff0000u);
  const float y0 = __uint_as_float(b << 16), y1 = __uint_as_float(b & 0xffff0000u);
  __nv_bfloat162 va = __floats2bfloat162_rn(fmaf(x0, cs0.x, y0 * cs0.y), fmaf(x1, cs1.x, y1 * cs1.y));
  __nv_bfloat162 vb = __floats2bfloat162_rn(fmaf(y0, cs0.x, -x0 * cs0.y), fmaf(y1, cs1.x, -x1 * cs1.y));
  a = *reinterpret_cast<uint32_t *>(&va);
  b = *reinterpret_cast<uint32_t *>(&vb);
}
// One thread rotates one row of a query tile (row r = TMEM lane r = the row whose softmax the
// thread computes).  The (cos, sin) values of the block are the same for every row: `cs` points
// to a copy of them in shared memory, read as warp-wide broadcasts.  The row is loaded in full
// before the arithmetic starts, so that the shared-memory latency is paid once.
template <int D>
__device__ __forceinline__ void rotate_q_row(const uint8_t *__restrict__ src, uint8_t *__restrict__ dst,
                                             const float2 *__restrict__ cs, int layout, int r) {
  constexpr int kRegion = 128 * 128;
  constexpr int kVec = D / 8;                      // 16-byte chunks per row
  const int rb = r * 128, sw = r & 7;
  uint4 v[kVec];
  int off[kVec];
#pragma unroll
  for (int i = 0; i < kVec; ++i) {
    off[i] = (i >> 3) * kRegion + rb + (((i & 7) ^ sw) << 4);     // chunk i of the row: columns 8 i .. 8 i + 7
    v[i] = *reinterpret_cast<const uint4 *>(src + off[i]);
  }
  if (layout == BA_ROPE_ADJACENT) {
#pragma unroll
    for (int i = 0; i < kVec; ++i) {
      const float4 c01 = *reinterpret_cast<const float4 *>(cs + i * 4);
      const float4 c23 = *reinterpret_cast<const float4 *>(cs + i * 4 + 2);
      v[i].x = rot_word_adjacent(v[i].x, make_float2(c01.x, c01.y)); v[i].y = rot_word_adjacent(v[i].y, make_float2(c01.z, c01.w));
      v[i].z = rot_word_adjacent(v[i].z, make_float2(c23.x, c23.y)); v[i].w = rot_word_adjacent(v[i].w, make_float2(c23.z, c23.w));
    }
  } else {
    // pairs (m, m + D/2): chunk i (< kVec / 2) holds x of pairs 8 i .. 8 i + 7, chunk i + kVec / 2 their partners
#pragma unroll
    for (int i = 0; i < kVec / 2; ++i) {
      const float4 *cp = reinterpret_cast<const float4 *>(cs + i * 8);
      const float4 c01 = cp[0], c23 = cp[1], c45 = cp[2], c67 = cp[3];
      uint4 &a = v[i], &b = v[i + kVec / 2];
      rot_words_half(a.x, b.x, make_float2(c01.x, c01.y), make_float2(c01.z, c01.w));
      rot_words_half(a.y, b.y, make_float2(c23.x, c23.y), make_float2(c23.z, c23.w));
      rot_words_half(a.z, b.z, make_float2(c45.x, c45.y), make_float2(c45.z, c45.w));
      rot_words_half(a.w, b.w, make_float2(c67.x, c67.y), make_float2(c67.z, c67.w));
    }
  }
#pragma unroll
  for (int i = 0; i < kVec; ++i) *reinterpret_cast<uint4 *>(dst + off[i]) = v[i];
}

// kFused selects the fused warm path at compile time, so that the plain path carries none of its code.
template <int D, bool kFused>
__global__ void __launch_bounds__(kThreads, 1)
ba_attend_sm100_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                       const __grid_constant__ CUtensorMap tmap_v, const __grid_constant__ CUtensorMap tmap_kc,
                       const __grid_constant__ CUtensorMap tmap_vc, const AttnParams p) {
  using L = Layout<D>;
  // setmaxnreg is a warpgroup-wide instruction: the four service warps (8-11) must ask for the same count
  constexpr int kServiceRegs = kFused ? kServiceRegsFused : kServiceRegsPlain;
  constexpr int kSoftmaxRegs = kFused ? kSoftmaxRegsFused : kSoftmaxRegsPlain;
  constexpr int kProdRegs = kServiceRegs, kMmaRegs = kServiceRegs, kSpareRegs = kServiceRegs;
  extern __shared__ uint8_t smem_raw[];
  uint8_t *smem = reinterpret_cast<uint8_t *>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Ctrl *ctrl = reinterpret_cast<Ctrl *>(smem + L::kCtrl);

  // inconsistent tables: no attention work is taken, a background job still runs
  const bool tables_ok = __ldg(p.seg.totals + 7) == BA_TABLES_VALID;
  const int tid = threadIdx.x, warp = tid >> 5;

  if (tid == 0) {
    for (int b = 0; b < 2; ++b) { mbar_init(&ctrl->q_full[b][0], 1); mbar_init(&ctrl->q_full[b][1], 1); mbar_init(&ctrl->q_empty[b], 1); }
    for (int s = 0; s < kStages; ++s) { mbar_init(&ctrl->kv_full[s], 1); mbar_init(&ctrl->kv_empty[s], 1); }
    for (int t = 0; t < 2; ++t) {
      mbar_init(&ctrl->s_full[t], 1); mbar_init(&ctrl->p_full[t][0], 128); mbar_init(&ctrl->p_full[t][1], 128);
      mbar_init(&ctrl->o_done[t], 1); mbar_init(&ctrl->o_free[t], 128);
      mbar_init(&ctrl->qr_full[t][0], 4); mbar_init(&ctrl->qr_full[t][1], 4); mbar_init(&ctrl->cs_full[t], D / 2);
      mbar_init(&ctrl->qraw_full[t], 1);
    }
    for (int k = 0; k < kWorkSlots; ++k) { mbar_init(&ctrl->work_full[k], 1); mbar_init(&ctrl->work_empty[k], 9); }
    ctrl->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 9) { tmem_alloc(&ctrl->tmem_base, 512); tmem_relinquish(); }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = ctrl->tmem_base;
  volatile int *abort_flag = &ctrl->abort_flag;

  // The CTA is persistent: its producer thread draws entries of the global work list from an
  // atomic counter (heaviest items first, whichever SM is free takes the next) and publishes them
  // to the other roles through a small ring; mbarrier phases simply keep counting across items, so the producer and the MMA warp run ahead into the next item while
  // the softmax warps still write out the previous one.
  // The softmax warps keep a whole 128-column row in registers; the service warps (8-11) need few.
  if (warp == 8) {
    // ------------------------------------------------------------ TMA producer
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kProdRegs));
    // balanced launch, a CTA that shares the front key tiles: prefix sum of the front tiles of every item (the
    // same for every head chunk), one item per lane, kept in shared memory for the scheduling thread
    int *bal_cu = reinterpret_cast<int *>(smem + L::kCtrl + kBalTableOff);
    int bal_np = 0;
    if (p.balanced && tables_ok) {
      bal_np = __ldg(p.seg.totals + 3);
      if (bal_np < 1 || bal_np > kBalMaxPairs || bal_np * p.n_chunks != p.balanced) {
        ba_record_status(p.status, BA_ERR_SHAPE);          // the tables describe another launch than the host sized
        bal_np = 0;
      } else if ((int)blockIdx.x >= p.balanced) {
        const int lane = tid & 31;
        int carry = 0;
        for (int base = 0; base < bal_np; base += 32) {
          const int i = base + lane;
          int x = 0;
          Item it;
          if (i < bal_np && resolve_item(p, bal_np - 1 - i, find_unit(p, bal_np - 1 - i), it)) x = max(0, it.n_tiles - p.bal_len);
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, o);
            if (lane >= o) x += y;
          }
          if (i < bal_np) bal_cu[i + 1] = carry + x;
          carry += __shfl_sync(0xffffffffu, x, 31);
        }
        if (lane == 0) bal_cu[0] = 0;
        __syncwarp();
      }
    }
    if (elect_one()) {
      prefetch_tmap(&tmap_q); prefetch_tmap(&tmap_k); prefetch_tmap(&tmap_v);
      prefetch_tmap(&tmap_kc); prefetch_tmap(&tmap_vc);
      // balanced launch: run [bal_pos, bal_end) of the front tiles of all (chunk, item), bal_hm of them per chunk
      int bal_pos = 0, bal_end = 0, bal_hm = 0, bal_nh = 0;
      long long bal_all = 0;
      if (bal_np > 0 && (int)blockIdx.x >= p.balanced) {
        bal_hm = bal_cu[bal_np];
        bal_all = (long long)bal_hm * p.n_chunks;
        bal_nh = (int)gridDim.x - p.balanced;
        const int j = (int)blockIdx.x - p.balanced;
        bal_pos = (int)(bal_all * j / bal_nh);
        bal_end = (int)(bal_all * (j + 1) / bal_nh);
      }
      auto balanced_entry = [&](int n_done) -> WorkEntry {
        WorkEntry e = {-1, -1, 0, 0, 0, 0, 0};
        if (bal_np == 0) return e;
        const int b = (int)blockIdx.x;
        if (b < p.balanced) {                              // the last bal_len key tiles of item b
          if (n_done > 0) return e;
          Item it;
          const int pair = bal_np - 1 - b % bal_np;
          e.unit = find_unit(p, pair);
          if (!resolve_item(p, pair, e.unit, it)) return e;
          e.pair = pair; e.chunk = b / bal_np;
          e.tile0 = max(0, it.n_tiles - p.bal_len);
          e.n_tiles = it.n_tiles - e.tile0;
          e.split = 0;
          e.fill = e.tile0 == 0 ? 1 : p.n_splits;           // nothing in front: the other slots stay empty
          return e;
        }
        if (bal_pos >= bal_end) return e;
        const int chunk = bal_pos / bal_hm, r = bal_pos - chunk * bal_hm;
        int lo = 0, hi = bal_np + 1;                        // item i with bal_cu[i] <= r < bal_cu[i + 1]
        while (lo < hi) { const int mid = (lo + hi) >> 1; if (bal_cu[mid] <= r) lo = mid + 1; else hi = mid; }
        const int i = lo - 1;
        const int front_end = chunk * bal_hm + bal_cu[i + 1];
        const int n = min(bal_end, front_end) - bal_pos;
        // the slot counts the CTAs from the one that holds the first front tile of the item
        const long long g0 = (long long)chunk * bal_hm + bal_cu[i];
        const int j_first = (int)(((g0 + 1) * bal_nh - 1) / bal_all);
        e.split = 1 + ((int)blockIdx.x - p.balanced) - j_first;
        if (e.split >= p.n_splits) { ba_record_status(p.status, BA_ERR_SHAPE); return e; }
        e.pair = bal_np - 1 - i; e.chunk = chunk;
        e.unit = find_unit(p, e.pair);
        e.tile0 = r - bal_cu[i]; e.n_tiles = n;
        e.fill = bal_pos + n == front_end ? e.split + 1 : p.n_splits;
        bal_pos += n;
        return e;
      };
      int gidx = 0;                       // K/V tiles requested so far (ring position)
      int n_items = 0;                    // items with at least one tile so far
      bool ok = true;
      Work wk;
      int n_work = 0;                    // work entries published so far
      for (;;) {
        // scheduler: take the next entry of the global work list and publish it to the other roles
        const int slot = n_work & (kWorkSlots - 1);
        ok = mbar_wait(&ctrl->work_empty[slot], ((n_work / kWorkSlots) & 1) ^ 1, abort_flag);
        if (!ok) break;
        // balanced launch: the next piece of this CTA's share; persistent launch: next entry of the global list;
        // one-item launch: this CTA's own entry, then stop
        WorkEntry e = {-1, -1, 0, 0, 0, 0, 0};
        if (tables_ok) {
          if (p.balanced) e = balanced_entry(n_work);
          else if (p.persistent) e = list_entry(p, atomicAdd(p.counters, 1));
          else if (n_work == 0) e = list_entry(p, (int)blockIdx.x);
        }
        const bool more = load_work(p, e, wk);
        if (!more) e.pair = -1;
        ctrl->work_ring[slot] = e;
        mbar_arrive(&ctrl->work_full[slot]);
        ++n_work;
        if (!more) break;
        if (wk.n_tiles == 0) continue;
        const Item &it = wk.it;
        if (!kFused) {      // (on the fused path the softmax warps fetch the query tiles themselves)
          // the Q buffers are free once every QK^T of the previous item has completed
          const int qb = p.q_double ? (n_items & 1) : 0;           // buffer pair of this entry
          const int q_use = p.q_double ? (n_items >> 1) : n_items;  // earlier entries that used it
          ok = mbar_wait(&ctrl->q_empty[qb], (q_use & 1) ^ 1, abort_flag);
          if (!ok) break;
          ++n_items;
          for (int t = 0; t < 2; ++t) {
            if (t >= it.n_qt) { mbar_arrive(&ctrl->q_full[qb][t]); continue; }   // (every entry moves both barriers on)
            mbar_arrive_expect_tx(&ctrl->q_full[qb][t], L::kTileBytes);
            uint8_t *dst = smem + (qb ? L::kBg + t * L::kTileBytes : (t ? L::kQ1 : L::kQ0));
            for (int c = 0; c < L::kChunks; ++c)
              tma_load_3d(dst + c * L::kRegionBytes, &tmap_q, &ctrl->q_full[qb][t], c * 64, wk.head0,
                          it.q_row0 + t * p.tok);
          }
        }
        // walk mode: cached keys are taken block by block (block pc, row offset poff inside it).  The
        // current block's length and first rows sit in registers and the next block's are fetched a
        // whole block ahead, so that no tile waits for a table look-up.
        int pc = 0, poff = 0;
        int c_len = 0, k_base = 0, v_base = 0, n_len = 0, n_kbase = 0, n_vbase = 0;
        // (for a paged operand the "base" of a block is the start of its page list)
        auto load_block = [&](int b, int &len, int &kb, int &vb) {
          if (b >= p.seg.n_cached_blocks) return;
          const int c0 = __ldg(p.seg.cache_cu + b);
          len = __ldg(p.seg.cache_cu + b + 1) - c0;
          const int pg = p.page_cu ? __ldg(p.page_cu + b) : 0;
          kb = p.k_paged ? pg : (p.k_src_off ? __ldg(p.k_src_off + b) : c0);
          vb = p.v_paged ? pg : (p.v_src_off ? __ldg(p.v_src_off + b) : c0);
        };
        if (p.walk && wk.tile0 < it.n_cache_tiles) {
          const int target = it.ctile0 + wk.tile0;
          pc = find_cache_block(p, it, target);
          poff = (target - __ldg(p.seg.cache_tile_cu + pc)) * kBlockN;
          load_block(pc, c_len, k_base, v_base);
          load_block(pc + 1, n_len, n_kbase, n_vbase);
        }
        // one 128-row tile of a paged operand: a box per page (pages of 128 rows or more hold whole tiles).
        // Parts of the tile past the end of the block are fetched from the block's last page: they are
        // masked, but what the tensor core multiplies by zero must still be finite.
        auto load_paged_tile = [&](uint8_t *dst, const CUtensorMap *m, uint64_t *bar, int list0, int off, int len) {
          const int page_rows = 1 << p.page_lg;
          const int sub_rows = min(kBlockN, page_rows), n_sub = kBlockN / sub_rows;
          const int last_page = (len - 1) >> p.page_lg;
          for (int sb = 0; sb < n_sub; ++sb) {
            const int t0 = off + sb * sub_rows;
            const int page = min(t0 >> p.page_lg, last_page);
            const int row = (__ldg(p.page_idx + list0 + page) << p.page_lg) + (t0 & (page_rows - 1));
            for (int c = 0; c < L::kChunks; ++c)
              tma_load_3d(dst + c * L::kRegionBytes + sb * sub_rows * 128, m, bar, c * 64, wk.kv_head, row);
          }
        };
        for (int j = 0; j < wk.n_tiles && ok; ++j) {
          const int jt = wk.tile0 + j;
          const bool cached = jt < it.n_cache_tiles;
          int k_row, v_row, t_off = 0, t_len = 0, t_kbase = 0, t_vbase = 0;
          bool k_pg = false, v_pg = false;
          if (!cached) {
            k_row = v_row = it.own_row0 + (jt - it.n_cache_tiles) * kBlockN;
          } else if (!p.walk) {
            k_row = v_row = it.cache_row0 + jt * kBlockN;
          } else {
            k_row = k_base + poff;
            v_row = v_base + poff;
            k_pg = p.k_paged; v_pg = p.v_paged;
            t_off = poff; t_len = c_len; t_kbase = k_base; t_vbase = v_base;
            ctrl->tile_valid[(gidx >> 1) & 7] = min(kBlockN, c_len - poff);   // read by the softmax warps
            poff += kBlockN;
            if (poff >= c_len) {
              ++pc; poff = 0;
              c_len = n_len; k_base = n_kbase; v_base = n_vbase;
              load_block(pc + 1, n_len, n_kbase, n_vbase);
            }
          }
          for (int kv = 0; kv < 2; ++kv) {
            const int stage = gidx % kStages;
            ok = mbar_wait(&ctrl->kv_empty[stage], ((gidx / kStages) & 1) ^ 1, abort_flag);
            if (!ok) break;
            const CUtensorMap *m = cached ? (kv ? &tmap_vc : &tmap_kc) : (kv ? &tmap_v : &tmap_k);
            uint8_t *dst = smem + L::kRing + stage * L::kTileBytes;
            mbar_arrive_expect_tx(&ctrl->kv_full[stage], L::kTileBytes);
            if (kv ? v_pg : k_pg) {
              load_paged_tile(dst, m, &ctrl->kv_full[stage], kv ? t_vbase : t_kbase, t_off, t_len);
            } else {
              for (int c = 0; c < L::kChunks; ++c)
                tma_load_3d(dst + c * L::kRegionBytes, m, &ctrl->kv_full[stage], c * 64, wk.kv_head, kv ? v_row : k_row);
            }
            ++gidx;
          }
        }
      }
      if (!ok) {
        // leave no copy in flight: wait (bounded) for the tiles already requested
        for (int idx = max(0, gidx - kStages); idx < gidx; ++idx)
          for (uint32_t spin = 0; spin < (1u << 20); ++spin)
            if (mbar_try_wait(&ctrl->kv_full[idx % kStages], (idx / kStages) & 1)) break;
      }
    }
  } else if (warp == 9) {
    // ------------------------------------------------------------ MMA issuer
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kMmaRegs));
    if (elect_one()) {
      const uint32_t tS[2] = {tmem, tmem + 128};
      const uint32_t tO[2] = {tmem + 256, tmem + 384};
      constexpr uint32_t idesc_qk = make_idesc_bf16(128, kBlockN, 0);
      constexpr uint32_t idesc_qk_half = make_idesc_bf16(128, kBlockN / 2, 0);   // keys 0..63 of the tile only
      constexpr uint32_t idesc_pv = make_idesc_bf16(128, D, 1);
      const uint32_t q_addr[2] = {smem_u32(smem + L::kQ0), smem_u32(smem + L::kQ1)};
      const uint32_t ring = smem_u32(smem + L::kRing);
      bool ok = true;
      auto wait_kv = [&](int idx) { return mbar_wait(&ctrl->kv_full[idx % kStages], (idx / kStages) & 1, abort_flag); };
      // descriptors differ only in their start-address field: build them once, add offsets (>> 4)
      const uint64_t q_desc[2] = {make_smem_desc(q_addr[0], 16, 1024), make_smem_desc(q_addr[1], 16, 1024)};
      const uint64_t k_desc0 = make_smem_desc(ring, 16, 1024);
      const uint64_t v_desc0 = make_smem_desc(ring, L::kRegionBytes, 1024);
      bool half_last = false;              // the entry's last key tile is used in its first 64 keys only
      int entry_tiles = 0;
      auto issue_qk_with = [&](int t, int jrel, int idx, uint64_t qd) {
        const uint64_t kd = k_desc0 + (uint64_t)(((idx % kStages) * L::kTileBytes) >> 4);
        const uint32_t idesc = (half_last && jrel + 1 == entry_tiles) ? idesc_qk_half : idesc_qk;
#pragma unroll
        for (int k = 0; k < D / 16; ++k) {
          const uint64_t off = (uint64_t)(((k >> 2) * L::kRegionBytes + (k & 3) * 32) >> 4);
          mma_ss(tS[t], qd + off, kd + off, idesc, k > 0);
        }
        mma_commit(&ctrl->s_full[t]);
      };
      // half = 0: keys 0..63 of the tile, half = 1: keys 64..127
      auto issue_pv = [&](int t, int idx, bool first, int half) {
        const uint64_t vd = v_desc0 + (uint64_t)(((idx % kStages) * L::kTileBytes) >> 4);
#pragma unroll
        for (int k = half * 4; k < half * 4 + 4; ++k)
          mma_ts(tO[t], tS[t] + k * 8, vd + (uint64_t)((k * 2048) >> 4), idesc_pv, (!first || k > 0) ? 1u : 0u);
      };
      int gidx = 0;                        // K/V tiles consumed so far (ring position)
      int q_uses[2] = {0, 0};              // items in which query tile t was loaded
      int p_uses[2] = {0, 0};              // P tiles of query tile t consumed
      Work wk = {};
      int n_work = 0;
      // Every loop over the query tile t below is unrolled, so that t is a constant and the small
      // per-tile arrays live in registers: this thread's issue latency is on the critical path.
      // fused path: a "version" of query tile t is the tile prepared for one key range of the entry --
      // rotated for one cached block, or plain for the final block's own keys.  The softmax threads
      // prepare versions in order into alternating buffers; both sides count them alike.
      const uint64_t qb_desc[2] = {make_smem_desc(smem_u32(smem + L::kBg), 16, 1024),         // second buffers
                                   make_smem_desc(smem_u32(smem + L::kBg + L::kTileBytes), 16, 1024)};
      int n_ver[2] = {0, 0};               // versions of query tile t taken so far
      int ver_end[2] = {-1, -1};           // the current version of tile t serves cached key tiles below this index
      int walk_pc = 0, walk_end = -1;      // block of the current cached tile and the tile index where it ends
      int cached_end = 0;                  // tiles [tile0, cached_end) of the entry are cached keys
      int q_buf = 0;                       // plain path: buffer pair that holds the entry's query tiles
      // S_t = Q_t K^T for tile `jrel` of the entry, whose keys sit at ring position idx
      auto issue_qk = [&](int t, int jrel, int idx) -> bool {
        if (!kFused) { issue_qk_with(t, jrel, idx, q_buf ? qb_desc[t] : q_desc[t]); return true; }
        const int jt = wk.tile0 + jrel;
        bool change = false;
        if (jt < cached_end) {
          const int g = wk.it.ctile0 + jt;
          if (g >= ver_end[t]) {                           // first key tile of another cached block
            if (walk_end < 0) { walk_pc = find_cache_block(p, wk.it, g); walk_end = __ldg(p.seg.cache_tile_cu + walk_pc + 1); }
            while (g >= walk_end) { ++walk_pc; walk_end = __ldg(p.seg.cache_tile_cu + walk_pc + 1); }
            ver_end[t] = walk_end;
            change = true;
          }
        } else if (ver_end[t] != 0x7fffffff) {             // first of the final block's own key tiles
          ver_end[t] = 0x7fffffff;
          change = true;
        }
        if (change) {
          BA_TR(5, n_ver[t] & 63, t * 2);
          if (!mbar_wait(&ctrl->qr_full[t][n_ver[t] & 1], (n_ver[t] >> 1) & 1, abort_flag)) return false;
          BA_TR(5, n_ver[t] & 63, t * 2 + 1);
          ++n_ver[t];
          tc_fence_after();
        }
        issue_qk_with(t, jrel, idx, ((n_ver[t] - 1) & 1) ? qb_desc[t] : q_desc[t]);
        return true;
      };
      for (;;) {
        const int slot = n_work & (kWorkSlots - 1);
        ok = mbar_wait(&ctrl->work_full[slot], (n_work / kWorkSlots) & 1, abort_flag);
        if (!ok) break;
        const WorkEntry e = ctrl->work_ring[slot];
        ++n_work;
        if (!load_work(p, e, wk)) break;
        mbar_arrive(&ctrl->work_empty[slot]);          // the entry has been decoded into registers
        const int n_tiles = wk.n_tiles, n_qt = wk.it.n_qt;
        if (n_tiles == 0) continue;
        half_last = last_tile_is_half(wk);
        entry_tiles = n_tiles;
        walk_end = -1; ver_end[0] = ver_end[1] = -1;
        cached_end = min(wk.tile0 + n_tiles, wk.it.n_cache_tiles);
        if (!kFused) {
          // (query tile 0 is part of every entry: q_uses[0] counts the entries)
          q_buf = p.q_double ? (q_uses[0] & 1) : 0;
          const int q_use = p.q_double ? (q_uses[0] >> 1) : q_uses[0];
#pragma unroll
          for (int t = 0; t < 2; ++t)
            if (t < n_qt && ok) ok = mbar_wait(&ctrl->q_full[q_buf][t], q_use & 1, abort_flag);
        }
        if (ok) ok = wait_kv(gidx);
        if (!ok) break;
        tc_fence_after();
#pragma unroll
        for (int t = 0; t < 2; ++t)
          if (t < n_qt && ok) ok = issue_qk(t, 0, gidx);
        if (!ok) break;
        mma_commit(&ctrl->kv_empty[gidx % kStages]);
        if (n_tiles == 1) mma_commit(&ctrl->q_empty[q_buf]);
        for (int j = 0; j < n_tiles && ok; ++j) {
          const bool last = j + 1 == n_tiles;
          const int iv = gidx + 2 * j + 1, ik = gidx + 2 * j + 2;   // ring positions of V_j and K_(j+1)
          BA_TR(3, j, 0);
          ok = wait_kv(iv);
          BA_TR(3, j, 1);
#pragma unroll
          for (int t = 0; t < 2; ++t) {
            if (t >= n_qt || !ok) continue;
            BA_TR(2, j, t * 4 + 0);
            // the first PV of an item overwrites O_t: the previous item's rows must have been read out
            if (j == 0) { ok = mbar_wait(&ctrl->o_free[t], (q_uses[t] & 1) ^ 1, abort_flag); if (!ok) continue; }
            ok = mbar_wait(&ctrl->p_full[t][0], p_uses[t] & 1, abort_flag);
            if (!ok) continue;
            tc_fence_after();
            BA_TR(2, j, t * 4 + 1);
            issue_pv(t, iv, j == 0, 0);
            // K_(j+1) is needed right after the second half of PV: make sure of it while P is still
            // being finished, off the critical path
            if (t == 0 && !last) { BA_TR(3, j, 2); ok = wait_kv(ik); if (!ok) continue; BA_TR(3, j, 3); }
            ok = mbar_wait(&ctrl->p_full[t][1], p_uses[t] & 1, abort_flag);
            if (!ok) continue;
            tc_fence_after();
            if (!(last && half_last)) issue_pv(t, iv, j == 0, 1);
            ++p_uses[t];
            BA_TR(2, j, t * 4 + 2);
            if (last) mma_commit(&ctrl->o_done[t]);
            if (t + 1 == n_qt) mma_commit(&ctrl->kv_empty[iv % kStages]);
            if (!last) {
              ok = issue_qk(t, j + 1, ik);
              if (!ok) continue;
              BA_TR(2, j, t * 4 + 3);
              if (t + 1 == n_qt) {
                mma_commit(&ctrl->kv_empty[ik % kStages]);
                if (j + 2 == n_tiles) mma_commit(&ctrl->q_empty[q_buf]);   // that was the item's last QK^T
              }
            }
          }
        }
        gidx += 2 * n_tiles;
#pragma unroll
        for (int t = 0; t < 2; ++t)
          if (t < n_qt) ++q_uses[t];
      }
    }
  } else if (warp >= 10) {
    // ------------------------------------------------------------ spare warps: background re-encoding
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kSpareRegs));
    if (p.bg.n_rows > 0) {
      // each spare warp runs the staged engine with its own two 16 KB stages; chunks are drawn from a
      // device-wide counter, so the job spreads over every CTA of the launch, early and late ones
      const int bw = warp - 10;
      ba_bg_smem *bsm = reinterpret_cast<ba_bg_smem *>(smem + L::kCtrl + 1024) + bw;
      if ((tid & 31) == 0) { mbar_init(&bsm->bar[0], 1); mbar_init(&bsm->bar[1], 1); fence_barrier_init(); }
      __syncwarp();
      ba_reencode_background(p.bg, p.counters + 1, smem + L::kBg + bw * 2 * kBgStageBytes, bsm, p.bg_rows_per_chunk,
                             p.status, [&](uint64_t *bar, uint32_t parity) { return mbar_wait(bar, parity, abort_flag); });
    }
  } else {
    // ------------------------------------------------------------ softmax, one thread per tile row
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    const int t = warp >> 2;
    const int r = tid & 127;
    const uint32_t lane_off = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t tS = tmem + t * 128 + lane_off;
    const uint32_t tO = tmem + 256 + t * 128 + lane_off;
    const float sl = p.scale_log2;
    int s_uses = 0;                       // S tiles of this query tile consumed so far
    int o_uses = 0;                       // items in which this query tile was active
    int n_staged = 0;                     // fused: (cos, sin) rows staged so far by this group
    int n_made = 0;                       // fused: versions of this query tile prepared so far
    int tiles_before = 0;                 // key tiles of all earlier items (the producer counts the same way)
    bool ok = true;
    Work wk;
    int n_work = 0;
    for (;;) {
      const int slot = n_work & (kWorkSlots - 1);
      ok = mbar_wait(&ctrl->work_full[slot], (n_work / kWorkSlots) & 1, abort_flag);
      if (!ok) break;
      const WorkEntry e = ctrl->work_ring[slot];
      ++n_work;
      if (!load_work(p, e, wk)) break;
      __syncwarp();
      if ((tid & 31) == 0) mbar_arrive(&ctrl->work_empty[slot]);   // one arrival per softmax warp
      const Item &it = wk.it;
      const int n_tiles = wk.n_tiles, tile0 = wk.tile0, head0 = wk.head0;
      const bool half_last = last_tile_is_half(wk);
      if (t < it.n_qt) {
      const int q_last = it.q_row0 + it.q_rows - 1;
      const int row_tok = it.q_row0 + t * p.tok + (r >> p.hpt_log2);
      // a row is stored only if it belongs to the item and lies inside the caller's tensors; tables that
      // describe more rows than the caller gave are reported, nothing is written past the end
      const bool row_valid = row_tok <= q_last && row_tok < p.n_q_rows;
      if (row_tok <= q_last && row_tok >= p.n_q_rows) ba_record_status(p.status, BA_ERR_SHAPE);
      const int tok_c = min(row_tok, q_last);               // rows past the block behave like its last row
      const int head = head0 + (r & (p.hpt - 1));
      float m_used = -INFINITY, l = 0.f;

      // fused path: this thread prepares row r of every version of query tile t (see the MMA warp):
      // the plain tile is fetched by the copy engine into the buffer the version will live in and, for a
      // cached block, every thread rotates its row there in place.  The first version of an entry is made on the spot; every later
      // one is begun after one tile of its predecessor and finished after the next, or at the latest
      // when its first key tile is next.
      const int tile_end = tile0 + n_tiles;
      const int cached_end = min(tile_end, it.n_cache_tiles);          // tiles [tile0, cached_end) are cached keys
      int f_pc = 0;                        // cached block of the version being prepared / in use
      int next_start = tile_end;           // first tile of the next version (tile_end: there is none)
      int prep = 0;                        // next version: 0 not begun, 1 row being fetched, 2 ready
      // The block's (cos, sin) row goes through shared memory: thread r < D/2 of the group holds
      // pair r, fetched one block ahead (cs_next), and the group's 128 threads wait for all of them.
      float2 *cs_stage = reinterpret_cast<float2 *>(smem + L::kCtrl + 1024) + t * 64;
      float2 cs_next = make_float2(1.f, 0.f);
      auto fetch_cs = [&](int pc) {
        if (r < D / 2 && pc < p.seg.n_cached_blocks) cs_next = __ldg(p.q_rope + (size_t)pc * (D / 2) + r);
      };
      auto ver_buf = [&](int v) { return smem + ((v & 1) ? L::kBg : L::kQ0) + t * L::kTileBytes; };
      auto begin_version = [&]() {       // plain query tile -> buffer of version n_made (one thread asks the copy engine)
        if (r == 0) {
          mbar_arrive_expect_tx(&ctrl->qraw_full[t], L::kTileBytes);
          for (int c = 0; c < L::kChunks; ++c)
            tma_load_3d(ver_buf(n_made) + c * L::kRegionBytes, &tmap_q, &ctrl->qraw_full[t], c * 64, head0,
                        it.q_row0 + t * p.tok);
        }
      };
      auto finish_version = [&](bool rotated) -> bool {
        if (!mbar_wait(&ctrl->qraw_full[t], n_made & 1, abort_flag)) return false;
        if (rotated) {
          if (r < D / 2) { cs_stage[r] = cs_next; mbar_arrive(&ctrl->cs_full[t]); }
          if (!mbar_wait(&ctrl->cs_full[t], n_staged & 1, abort_flag)) return false;
          ++n_staged;
          rotate_q_row<D>(ver_buf(n_made), ver_buf(n_made), cs_stage, p.rope_layout, r);
        }
        fence_proxy_async();                               // the tensor core reads through the async proxy
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(&ctrl->qr_full[t][n_made & 1]);
        ++n_made;
        return true;
      };
      // where the version after the one for block `pc` (or after the plain one: pc < 0) starts
      auto plan_next = [&](int pc) {
        next_start = tile_end;
        if (pc >= 0) {
          const int e = __ldg(p.seg.cache_tile_cu + pc + 1) - it.ctile0;   // first tile after the block
          if (e < tile_end) next_start = min(e, cached_end);
          if (next_start < cached_end) fetch_cs(pc + 1);
        }
        prep = 0;
      };
      if (kFused && n_tiles > 0) {
        const bool first_cached = tile0 < cached_end;
        if (first_cached) { f_pc = find_cache_block(p, it, it.ctile0 + tile0); fetch_cs(f_pc); }
        begin_version();
        ok = finish_version(first_cached);
        if (!ok) break;
        plan_next(first_cached ? f_pc : -1);
      }

      for (int j = 0; j < n_tiles; ++j) {
        if (r == 0) BA_TR(t, j, 0);
        ok = mbar_wait(&ctrl->s_full[t], s_uses & 1, abort_flag);
        if (!ok) break;
        ++s_uses;
        tc_fence_after();
        if (r == 0) BA_TR(t, j, 1);
        // visible columns of this tile for this row: 0 .. lim
        int lim;
        const int jt = tile0 + j;
        if (jt < it.n_cache_tiles) lim = p.walk ? ctrl->tile_valid[(tiles_before + j) & 7] - 1
                                                     : it.cache_len - jt * kBlockN - 1;
        else lim = tok_c - (it.own_row0 + (jt - it.n_cache_tiles) * kBlockN);
        uint64_t sum2[4] = {0ull, 0ull, 0ull, 0ull};       // packed (0.f, 0.f)
        // One tile of softmax for this row over kCols key columns: 128, or 64 for a half tile (only the first
        // 64 keys were multiplied; nothing of the second half is loaded, exponentiated or handed over).
        auto tile_softmax = [&](auto cols_tag) {
          constexpr int kCols = decltype(cols_tag)::value;
          uint32_t s[kCols];
#pragma unroll
          for (int c = 0; c < kCols / 32; ++c) tmem_ld_32x32b_x32(tS + c * 32, *reinterpret_cast<uint32_t(*)[32]>(&s[c * 32]));
          tmem_wait_ld();
          if (r == 0) BA_TR(t, j, 2);
          if (lim < kCols - 1) {
#pragma unroll
            for (int c = 0; c < kCols; ++c)
              if (c > lim) s[c] = 0xff800000u;               // -inf
          }
          // row maximum by a wide tree of three-input maxima (128 -> 43 -> 15 -> 5 -> 1)
          constexpr int n1 = (kCols + 2) / 3, n2 = (n1 + 2) / 3, n3 = (n2 + 2) / 3;
          float l1[n1], l2[n2], l3[n3];
          auto mx_at = [](const float *a, int n, int i) {    // max of a[3i], a[3i+1], a[3i+2] where they exist
            return (3 * i + 2 < n) ? max3(a[3 * i], a[3 * i + 1], a[3 * i + 2])
                                   : (3 * i + 1 < n) ? fmaxf(a[3 * i], a[3 * i + 1]) : a[3 * i];
          };
          const float *sf = reinterpret_cast<const float *>(s);
#pragma unroll
          for (int i = 0; i < n1; ++i) l1[i] = mx_at(sf, kCols, i);
#pragma unroll
          for (int i = 0; i < n2; ++i) l2[i] = mx_at(l1, n1, i);
#pragma unroll
          for (int i = 0; i < n3; ++i) l3[i] = mx_at(l2, n2, i);
          float mx = l3[0];
#pragma unroll
          for (int i = 1; i < n3; ++i) mx = fmaxf(mx, l3[i]);
          const float m_new = fmaxf(m_used, mx);
          if (r == 0) BA_TR(t, j, 3);
          if (j == 0) {
            m_used = m_new;
          } else {
            const bool grow = (m_new - m_used) * sl > kRescaleThreshold;
            if (__any_sync(0xffffffffu, grow)) {
              // 1 when this row's maximum did not move (also when the row has seen no key yet)
              const float alpha = (m_new == -INFINITY) ? 1.f : ex2((m_used - m_new) * sl);
              m_used = m_new;
              l *= alpha;
#pragma unroll
              for (int c = 0; c < D / 32; ++c) {
                uint32_t o[32];
                tmem_ld_32x32b_x32(tO + c * 32, o);
                tmem_wait_ld();
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                tmem_st_32x32b_x32(tO + c * 32, o);
              }
            }
          }
          const float neg_m = (m_used == -INFINITY) ? 0.f : -m_used * sl;   // no visible key so far: every p is 0
          const uint64_t sl2 = pack2(sl, sl), negm2 = pack2(neg_m, neg_m);
          // P is handed to the MMA warp in two halves so that PV can start on the first 64 keys
          // while the second 64 are still being exponentiated.  The arithmetic is packed fp32x2.  The
          // store of the first half completes while the second half is begun.
          constexpr int kLead = kCols > 64 ? 16 : 0;       // column pairs of the second half done before the first is handed over
          uint32_t pk[32], pk1[kCols > 64 ? 32 : 1];
          auto expo = [&](int e0, uint32_t &dst, int i) {
            const uint64_t x2 = fma2(pack2(__uint_as_float(s[e0]), __uint_as_float(s[e0 + 1])), sl2, negm2);
            float x0, x1;
            unpack2(x2, x0, x1);
            const float p0 = ex2(x0), p1 = ex2(x1);
            sum2[i & 3] = add2(sum2[i & 3], pack2(p0, p1));
            __nv_bfloat162 v = __floats2bfloat162_rn(p0, p1);
            dst = *reinterpret_cast<uint32_t *>(&v);
          };
#pragma unroll
          for (int i = 0; i < 32; ++i) expo(2 * i, pk[i], i);
          tmem_st_32x32b_x32(tS, pk);
#pragma unroll
          for (int i = 0; i < kLead; ++i) expo(64 + 2 * i, pk1[i], i);
          tmem_wait_st();
          tc_fence_before();
          mbar_arrive(&ctrl->p_full[t][0]);
          if (r == 0) BA_TR(t, j, 4);
          if constexpr (kCols > 64) {
#pragma unroll
            for (int i = kLead; i < 32; ++i) expo(64 + 2 * i, pk1[i], i);
            tmem_st_32x32b_x32(tS + 32, *reinterpret_cast<uint32_t(*)[32]>(&pk1[0]));
            tmem_wait_st();
            tc_fence_before();
          }
          mbar_arrive(&ctrl->p_full[t][1]);               // (half tile: nothing to hand over, that product is skipped)
          if (r == 0) BA_TR(t, j, 5);
        };
        if (half_last && j + 1 == n_tiles) tile_softmax(std::integral_constant<int, kBlockN / 2>{});
        else tile_softmax(std::integral_constant<int, kBlockN>{});
        // P of this tile is with the tensor core: time to work on the next version of the query row
        if (kFused && next_start < tile_end) {
          const bool due = tile0 + j + 1 == next_start;    // the next tile is the first to need it
          const bool next_cached = next_start < cached_end;
          if (r == 0) BA_TR(t, j, 6);
          if (prep == 0) { begin_version(); prep = 1; if (due) { ok = finish_version(next_cached); prep = 2; } }
          else if (prep == 1) { ok = finish_version(next_cached); prep = 2; }
          if (!ok) break;
          if (r == 0) BA_TR(t, j, 7);
          if (due) { if (next_cached) ++f_pc; plan_next(next_cached ? f_pc : -1); }
        }
        float sum[8];
#pragma unroll
        for (int i = 0; i < 4; ++i) unpack2(sum2[i], sum[2 * i], sum[2 * i + 1]);
        l += ((sum[0] + sum[1]) + (sum[2] + sum[3])) + ((sum[4] + sum[5]) + (sum[6] + sum[7]));
      }

      if (ok && n_tiles > 0) { ok = mbar_wait(&ctrl->o_done[t], o_uses & 1, abort_flag); ++o_uses; }
      if (ok) {
        tc_fence_after();
        const float inv = l > 0.f ? 1.f / l : 0.f;
        const float lse_val = l > 0.f ? (m_used * sl + log2f(l)) * 0.6931471805599453f : -INFINITY;
        const size_t orow = ((size_t)row_tok * p.Hq + head) * D;
        const bool partial = p.n_splits > 1;
        float *part = partial ? p.o_part + (size_t)wk.split * p.n_q_rows * p.Hq * D + orow : nullptr;
#pragma unroll
        for (int c = 0; c < D / 32; ++c) {
          uint32_t o[32];
          if (n_tiles > 0) {
            tmem_ld_32x32b_x32(tO + c * 32, o);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = 0u;
          }
          if (row_valid) {
            if (partial) {
              // 32-byte stores (the workspace is aligned for them): a thread owns a row, so each fills a whole sector
              float *dst = part + c * 32;
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                float v[8];
#pragma unroll
                for (int e = 0; e < 8; ++e) v[e] = __uint_as_float(o[8 * i + e]) * inv;
                st_global_v8(dst + 8 * i, v);
              }
            } else if (p.out_f32) {
              float4 *dst = reinterpret_cast<float4 *>(reinterpret_cast<float *>(p.o) + orow + c * 32);
#pragma unroll
              for (int i = 0; i < 8; ++i)
                dst[i] = make_float4(__uint_as_float(o[4 * i]) * inv, __uint_as_float(o[4 * i + 1]) * inv,
                                     __uint_as_float(o[4 * i + 2]) * inv, __uint_as_float(o[4 * i + 3]) * inv);
            } else {
              uint4 *dst = reinterpret_cast<uint4 *>(reinterpret_cast<__nv_bfloat16 *>(p.o) + orow + c * 32);
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                uint32_t w[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  __nv_bfloat162 v = __floats2bfloat162_rn(__uint_as_float(o[8 * i + 2 * e]) * inv,
                                                           __uint_as_float(o[8 * i + 2 * e + 1]) * inv);
                  w[e] = *reinterpret_cast<uint32_t *>(&v);
                }
                dst[i] = make_uint4(w[0], w[1], w[2], w[3]);
              }
            }
          }
        }
        if (n_tiles > 0) {
          // O_t has been read out of tensor memory: the next item's first PV may overwrite it
          tc_fence_before();
          mbar_arrive(&ctrl->o_free[t]);
        }
        if (row_valid) {
          if (partial) {
            p.lse_part[((size_t)wk.split * p.n_q_rows + row_tok) * p.Hq + head] = lse_val;
            for (int s = wk.fill; s < p.n_splits; ++s)      // slots no entry of this item writes: empty
              p.lse_part[((size_t)s * p.n_q_rows + row_tok) * p.Hq + head] = -INFINITY;
          } else if (p.lse) p.lse[(size_t)row_tok * p.Hq + head] = lse_val;
        }
      }
      }
      tiles_before += n_tiles;
    }
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0) {
    if (ctrl->abort_flag) ba_record_status(p.status, BA_ERR_TIMEOUT);
    if (p.counters) {
      // every role of this CTA is done with the counters; the CTA that finishes last puts them back to zero
      __threadfence();
      if (atomicAdd(p.counters + 2, 1) == (int)gridDim.x - 1) {
        p.counters[0] = 0; p.counters[1] = 0;
        __threadfence();
        p.counters[2] = 0;
      }
    }
  }
  if (warp == 9) tmem_dealloc(tmem, 512);
}

// Merge of split-KV partial results: o = sum_s w_s o_s / sum_s w_s with w_s = exp(lse_s - max lse).
// One thread per 4 output columns; the order of the sum is fixed, so results are run-to-run stable.
// kNS > 0: the number of splits is known at compile time and every load is issued before the first use.
template <int D, int kNS>
__global__ void __launch_bounds__(256)
ba_combine_splits_kernel(const float *__restrict__ o_part, const float *__restrict__ lse_part, void *o, float *lse,
                         int n_rows_heads, int n_splits, int out_f32) {
  const int idx = blockIdx.x * blockDim.x + threadIdx.x;
  constexpr int kVec = D / 4;
  const int rh = idx / kVec, v = idx - rh * kVec;
  if (rh >= n_rows_heads) return;
  float den = 0.f, mx = -INFINITY;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (kNS > 0) {
    float ls[kNS > 0 ? kNS : 1];
    float4 x[kNS > 0 ? kNS : 1];
#pragma unroll
    for (int s = 0; s < kNS; ++s) {
      ls[s] = __ldg(lse_part + (size_t)s * n_rows_heads + rh);
      x[s] = __ldcs(reinterpret_cast<const float4 *>(o_part + ((size_t)s * n_rows_heads + rh) * D) + v);
    }
#pragma unroll
    for (int s = 0; s < kNS; ++s) mx = fmaxf(mx, ls[s]);
#pragma unroll
    for (int s = 0; s < kNS; ++s) {
      const float w = (ls[s] == -INFINITY) ? 0.f : __expf(ls[s] - mx);
      if (w == 0.f) x[s] = make_float4(0.f, 0.f, 0.f, 0.f);   // an empty slot holds no values at all
      den += w;
      acc.x = fmaf(w, x[s].x, acc.x); acc.y = fmaf(w, x[s].y, acc.y); acc.z = fmaf(w, x[s].z, acc.z); acc.w = fmaf(w, x[s].w, acc.w);
    }
  } else {
    for (int s = 0; s < n_splits; ++s) mx = fmaxf(mx, __ldg(lse_part + (size_t)s * n_rows_heads + rh));
    for (int s = 0; s < n_splits; ++s) {
      const float ls = __ldg(lse_part + (size_t)s * n_rows_heads + rh);
      const float w = (ls == -INFINITY) ? 0.f : __expf(ls - mx);
      float4 x = __ldg(reinterpret_cast<const float4 *>(o_part + ((size_t)s * n_rows_heads + rh) * D) + v);
      if (w == 0.f) x = make_float4(0.f, 0.f, 0.f, 0.f);
      den += w;
      acc.x = fmaf(w, x.x, acc.x); acc.y = fmaf(w, x.y, acc.y); acc.z = fmaf(w, x.z, acc.z); acc.w = fmaf(w, x.w, acc.w);
    }
  }
  const float inv = 1.f / den;
  acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
  if (out_f32) {
    reinterpret_cast<float4 *>(reinterpret_cast<float *>(o) + (size_t)rh * D)[v] = acc;
  } else {
    __nv_bfloat162 a = __floats2bfloat162_rn(acc.x, acc.y), b = __floats2bfloat162_rn(acc.z, acc.w);
    uint2 w2 = make_uint2(*reinterpret_cast<uint32_t *>(&a), *reinterpret_cast<uint32_t *>(&b));
    reinterpret_cast<uint2 *>(reinterpret_cast<__nv_bfloat16 *>(o) + (size_t)rh * D)[v] = w2;
  }
  if (lse && v == 0) lse[rh] = mx + logf(den);
}

// ------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                  const cuuint64_t *, const cuuint32_t *, const cuuint32_t *,
                                  CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                  CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void *p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [rows, heads, d] bf16 viewed as a 3-D tensor (d, head, row); box = 64 columns x box_heads x box_rows, 128-byte swizzle.
bool make_map(CUtensorMap *m, const void *ptr, int D, int heads, long long rows, int box_heads, int box_rows) {
  EncodeTiledFn enc = encode_fn();
  if (!enc || rows < 1) return false;
  cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)heads * D * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
  cuuint32_t es[3] = {1, 1, 1};
  return enc(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(ptr), dims, strides, box, es,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Tensor maps of the tensors recently passed to the attention calls.  A serving loop hands the same
// few buffers to the library layer after layer; encoding a map costs a driver call each time, so
// the maps are kept in a small direct-mapped table keyed by everything that goes into them.
struct ba_map_cache {
  static constexpr int kSlots = 512;
  struct Slot {
    const void *ptr;
    long long rows;
    int D, heads, box_heads, box_rows;
    alignas(64) CUtensorMap map;
  } slot[kSlots];
};

namespace {

const CUtensorMap *cached_map(ba_ctx *ctx, const void *ptr, int D, int heads, long long rows, int box_heads,
                              int box_rows) {
  uint64_t h = (uint64_t)(uintptr_t)ptr * 0x9E3779B97F4A7C15ull;
  h ^= (uint64_t)rows * 0xC2B2AE3D27D4EB4Full + (uint64_t)(box_heads * 131 + box_rows);
  ba_map_cache::Slot &sl = ctx->maps->slot[(h >> 40) & (ba_map_cache::kSlots - 1)];
  if (sl.ptr == ptr && sl.rows == rows && sl.D == D && sl.heads == heads && sl.box_heads == box_heads &&
      sl.box_rows == box_rows)
    return &sl.map;
  sl.ptr = nullptr;
  if (!make_map(&sl.map, ptr, D, heads, rows, box_heads, box_rows)) return nullptr;
  sl.ptr = ptr; sl.rows = rows; sl.D = D; sl.heads = heads; sl.box_heads = box_heads; sl.box_rows = box_rows;
  return &sl.map;
}

template <int D>
constexpr int attend_smem_bytes() {
  // ask for more than half of the SM's shared memory so that two CTAs never share an SM
  // (each CTA allocates all 512 tensor-memory columns)
  return Layout<D>::kBytes + 1024 > 120 * 1024 ? Layout<D>::kBytes + 1024 : 120 * 1024;
}

}  // namespace

// Per-context set-up of the attention path, with the context's device current: the kernels' shared-memory
// limit is raised once here instead of on every launch, and the tensor-map table is created.
ba_status ba_attend_sm100_setup(ba_ctx *ctx) {
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_attend_sm100_kernel<128, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   attend_smem_bytes<128>()));
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_attend_sm100_kernel<128, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   attend_smem_bytes<128>()));
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_attend_sm100_kernel<64, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   attend_smem_bytes<64>()));
  BA_CUDA_TRY(cudaFuncSetAttribute(ba_attend_sm100_kernel<64, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                   attend_smem_bytes<64>()));
  ctx->maps = new (std::nothrow) ba_map_cache();
  if (!ctx->maps) return BA_ERR_CUDA;
  for (auto &sl : ctx->maps->slot) sl.ptr = nullptr;
  return BA_OK;
}

void ba_attend_sm100_teardown(ba_ctx *ctx) {
  delete ctx->maps;
  ctx->maps = nullptr;
}

// Diagnostic: one CTA waits on an mbarrier that nothing ever arrives on, with the same bounded
// wait the attention kernel uses, so the expiry path (abort flag, status word, clean return) can be
// checked on a live device without any fault.
__global__ void ba_wait_expiry_kernel(int32_t *status) {
  __shared__ uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) { mbar_init(&bar, 1); abort_flag = 0; fence_barrier_init(); }
  __syncthreads();
  const bool ok = mbar_wait(&bar, 0, &abort_flag);       // never completes: gives up after the poll limit
  __syncthreads();
  if (threadIdx.x == 0 && (!ok || abort_flag)) ba_record_status(status, BA_ERR_TIMEOUT);
}

extern "C" ba_status ba_selftest_wait_expiry(ba_ctx *ctx, void *stream) {
  if (!ctx) return BA_ERR_INVALID_ARG;
  BA_CUDA_TRY(cudaSetDevice(ctx->device));
  ba_wait_expiry_kernel<<<1, 64, 0, (cudaStream_t)stream>>>(ctx->dev_status);
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 1;
  return BA_OK;
}

// Heads of one KV group packed into a query tile: the largest of 4, 2, 1 that divides the group size.
int ba_heads_per_tile(const ba_config &c) {
  int G = c.n_q_heads / c.n_kv_heads;
  return (G % 4 == 0) ? 4 : (G % 2 == 0) ? 2 : 1;
}

ba_status ba_attend_sm100_launch(ba_ctx *ctx, const ba_attend_args &a, const ba_segments *seg,
                                 cudaStream_t stream) {
  const int D = ctx->cfg.head_dim, Hq = ctx->cfg.n_q_heads, Hkv = ctx->cfg.n_kv_heads;
  AttnParams p;
  p.o = a.o; p.lse = a.lse; p.status = ctx->dev_status; p.out_f32 = a.out_f32;
  p.Hq = Hq; p.Hkv = Hkv; p.G = Hq / Hkv;
  p.hpt = ba_heads_per_tile(ctx->cfg);
  p.hpt_log2 = p.hpt == 4 ? 2 : p.hpt == 2 ? 1 : 0;
  p.tok = 128 / p.hpt;
  p.scale = ctx->scale;
  p.scale_log2 = ctx->scale * 1.4426950408889634f;
  p.final_only = a.final_only;
  p.balanced = 0; p.bal_len = 0; p.q_double = 0;
  p.v_src_off = a.final_only ? a.v_src_off : nullptr;
  p.fused = a.final_only && a.fused && a.n_cache_rows > 0;
  p.k_src_off = p.fused ? a.k_src_off : nullptr;
  p.page_cu = nullptr; p.page_idx = nullptr; p.page_lg = 0; p.k_paged = 0; p.v_paged = 0;
  if (a.final_only && a.page_rows > 0 && a.n_cache_rows > 0) {
    p.page_cu = a.page_cu; p.page_idx = a.page_idx;
    while ((1 << p.page_lg) < a.page_rows) ++p.page_lg;
    p.v_paged = 1;
    p.k_paged = p.fused ? 1 : 0;
    p.v_src_off = nullptr; p.k_src_off = nullptr;
  }
  p.walk = p.v_src_off != nullptr || p.fused || p.v_paged;
  p.rope_layout = ctx->cfg.rope_layout;
  p.q_rope = p.fused ? reinterpret_cast<const float2 *>(seg->cache_rope) : nullptr;
  if (p.fused && !p.q_rope) return BA_ERR_INVALID_ARG;
  p.n_q_rows = a.n_q_rows;
  p.seg = *seg;
  if (seg->q_tile_tokens != 2 * p.tok) return BA_ERR_INVALID_ARG;

  // Split the keys of each work item over several CTAs when the items alone cannot fill the
  // GPU (a short final block over a long cache).  The split count minimises
  // waves x (tiles per CTA + a fixed per-CTA cost) and is capped by the workspace.
  const int pair_tok = 2 * p.tok;
  const int n_units = a.final_only ? seg->batch : seg->n_blocks;
  // work items: the exact count when ba_segment() saw the lengths on the host, else an upper bound
  const int pairs_known = a.final_only ? seg->n_final_items : seg->n_prompt_items;
  const unsigned pairs_upper = pairs_known > 0 ? (unsigned)pairs_known : (unsigned)(a.n_q_rows / pair_tok + n_units);
  const long long items = (long long)((a.n_q_rows + pair_tok - 1) / pair_tok) * (Hq / p.hpt);
  int n_splits = 1;
  if (a.final_only && items < 2LL * ctx->sm_count) {
    // key tiles of an average item: counted by ba_segment() when it saw the lengths, else estimated
    const int32_t *ft = seg->final_key_tiles + (p.walk ? 3 : 0);
    const long long avg_tiles = (ft[0] > 0 && seg->n_final_items > 0)
                                    ? (ft[0] + seg->n_final_items - 1) / seg->n_final_items
                                    : ((long long)a.n_cache_rows / seg->batch + pair_tok) / kBlockN + 1;
    const size_t per_split = (size_t)a.n_q_rows * Hq * (D + 1) * sizeof(float);
    // the angle table of a queued re-encoding job sits at the end of the workspace and is read by
    // this very launch: the partial results must stay below it
    const size_t taken = ba_scratch_offset(ctx) + ctx->pending_table_bytes;
    const size_t avail = ctx->workspace_bytes > taken ? ctx->workspace_bytes - taken : 0;
    const int cap = (int)min((size_t)32, per_split ? avail / per_split : 0);
    // equal splits or the balanced launch (ba_plan_splits, above the kernels' common declarations)
    const ba_split_plan plan = ba_plan_splits(ctx->sm_count, items, seg->n_final_items, Hq / p.hpt, avg_tiles, ft, cap);
    n_splits = plan.n_splits; p.balanced = plan.balanced; p.bal_len = plan.bal_len;
  }
  p.n_splits = n_splits;
  p.n_chunks = Hq / p.hpt;
  // More entries than SMs: persistent CTAs, one per SM, draw entries from a counter, which hides each
  // entry's start-up and write-out behind its neighbours (cold prefill: many entries per SM; final block
  // over a long cache: about two, the write-out of a CTA's first entry overlaps the start of its second).
  // Shorter lists are launched one CTA per entry.
  const long long work_upper = (long long)pairs_upper * (Hq / p.hpt) * n_splits;
  p.persistent = !p.balanced && items * n_splits > (a.final_only ? 1LL : 2LL) * ctx->sm_count;
  // the counters live in the last 256 bytes below the scratch area: zeroed by ba_create, left at zero by every launch
  int32_t *counters = nullptr;
  if (ctx->workspace && ctx->workspace_bytes >= ba_scratch_offset(ctx))
    counters = reinterpret_cast<int32_t *>(reinterpret_cast<char *>(ctx->workspace) + ba_scratch_offset(ctx) - 256);
  p.counters = nullptr;
  if (p.persistent && !counters) p.persistent = 0;   // a context without workspace: one CTA per entry, however many
  if (p.persistent) p.counters = counters;
  p.o_part = nullptr; p.lse_part = nullptr;
  if (n_splits > 1) {
    p.o_part = reinterpret_cast<float *>(reinterpret_cast<char *>(ctx->workspace) + ba_scratch_offset(ctx));
    p.lse_part = p.o_part + (size_t)n_splits * a.n_q_rows * Hq * D;
  }

  const CUtensorMap *mq = cached_map(ctx, a.q, D, Hq, a.n_q_rows, p.hpt, p.tok);
  const CUtensorMap *mk = cached_map(ctx, a.k, D, Hkv, a.n_kv_rows, 1, kBlockN);
  const CUtensorMap *mv = cached_map(ctx, a.v, D, Hkv, a.n_kv_rows, 1, kBlockN);
  if (!mq || !mk || !mv) return BA_ERR_CUDA;
  CUtensorMap tq = *mq, tk = *mk, tv = *mv, tkc = *mk, tvc = *mv;   // (a slot may be reused by a later look-up)
  if (a.final_only && a.n_cache_rows > 0) {
    const int page_box = p.v_paged ? min(kBlockN, a.page_rows) : kBlockN;
    const CUtensorMap *mkc = cached_map(ctx, a.k_cache, D, Hkv, p.fused ? a.n_k_rows : a.n_cache_rows, 1,
                                        p.k_paged ? page_box : kBlockN);
    if (!mkc) return BA_ERR_CUDA;
    tkc = *mkc;
    const CUtensorMap *mvc = cached_map(ctx, a.v_cache, D, Hkv, (a.v_src_off || p.v_paged) ? a.n_v_rows : a.n_cache_rows, 1,
                                        page_box);
    if (!mvc) return BA_ERR_CUDA;
    tvc = *mvc;
  }
  dim3 grid((unsigned)((p.persistent || p.balanced) ? ctx->sm_count : work_upper));
  // a queued re-encoding job rides along in the spare warps; a job whose rows do not fit the
  // staging buffers is run on its own first
  p.bg.n_rows = 0; p.bg_rows_per_chunk = 0;
  if (ctx->has_pending) {
    const int row_bytes = ctx->pending.row_vecs * 16;
    if (row_bytes <= kBgStageBytes && !p.fused && counters) {   // (the fused path has other uses for the spare warps' staging area)
      p.bg = ctx->pending;
      ctx->has_pending = 0;
      ctx->pending_table_bytes = 0;
      p.bg_rows_per_chunk = kBgStageBytes / row_bytes < 32 ? kBgStageBytes / row_bytes : 32;
      p.counters = counters;
    } else {
      ba_status fs = ba_flush_pending(ctx, stream);
      if (fs != BA_OK) return fs;
    }
  }
  p.q_double = (!p.fused && p.bg.n_rows == 0) ? 1 : 0;     // the staging area is free: second pair of query buffers
  // Side output of the fused call: the re-encoded keys, written by the stand-alone re-encoding kernel on the
  // context's side stream beside the attention launch (which cannot share an SM with anything and leaves
  // some SMs idle in its last wave); the caller's stream continues only when both are done.  (Measured
  // alternative: the spare warps of the attention CTAs moving the rows cost 50 us per layer at 32K context,
  // more than the kernel alone takes.)
  const bool side_job = p.fused && a.k_out;
  if (side_job) {
    ba_reencode_job job = ba_make_reencode_job(ctx, a.k_cache, a.k_src_off, a.n_k_rows, a.k_out, seg->cache_cu,
                                               seg->cache_delta, seg->n_cached_blocks, a.n_cache_rows,
                                               reinterpret_cast<const float2 *>(seg->cache_rope));
    if (p.k_paged) { job.src_off = nullptr; job.page_cu = a.page_cu; job.page_idx = a.page_idx; job.page_lg = p.page_lg; }
    BA_CUDA_TRY(cudaEventRecord(ctx->ev_fork, stream));
    BA_CUDA_TRY(cudaStreamWaitEvent(ctx->side_stream, ctx->ev_fork, 0));
    ba_status rs = ba_reencode_main_launch(ctx, job, ctx->side_stream);
    if (rs != BA_OK) return rs;
    BA_CUDA_TRY(cudaEventRecord(ctx->ev_join, ctx->side_stream));
  }
  if (D == 128) {
    auto kern = p.fused ? ba_attend_sm100_kernel<128, true> : ba_attend_sm100_kernel<128, false>;
    kern<<<grid, kThreads, attend_smem_bytes<128>(), stream>>>(tq, tk, tv, tkc, tvc, p);
  } else {
    auto kern = p.fused ? ba_attend_sm100_kernel<64, true> : ba_attend_sm100_kernel<64, false>;
    kern<<<grid, kThreads, attend_smem_bytes<64>(), stream>>>(tq, tk, tv, tkc, tvc, p);
  }
  BA_CUDA_TRY(cudaGetLastError());
  ctx->launches += 1;
  ctx->last_attend[0] = (int32_t)grid.x; ctx->last_attend[1] = n_splits;
  ctx->last_attend[2] = p.balanced; ctx->last_attend[3] = p.bal_len;
  if (side_job) BA_CUDA_TRY(cudaStreamWaitEvent(stream, ctx->ev_join, 0));
  if (n_splits > 1) {
    const int n_rh = a.n_q_rows * Hq;
    const long long threads = (long long)n_rh * (D / 4);
    const unsigned cgrid = (unsigned)((threads + 255) / 256);
    auto launch = [&](auto kern) {
      kern<<<cgrid, 256, 0, stream>>>(p.o_part, p.lse_part, a.o, a.lse, n_rh, n_splits, a.out_f32);
    };
    if (D == 128) {
      if (n_splits == 2) launch(ba_combine_splits_kernel<128, 2>);
      else if (n_splits == 3) launch(ba_combine_splits_kernel<128, 3>);
      else if (n_splits == 4) launch(ba_combine_splits_kernel<128, 4>);
      else launch(ba_combine_splits_kernel<128, 0>);
    } else {
      if (n_splits == 2) launch(ba_combine_splits_kernel<64, 2>);
      else if (n_splits == 3) launch(ba_combine_splits_kernel<64, 3>);
      else if (n_splits == 4) launch(ba_combine_splits_kernel<64, 4>);
      else launch(ba_combine_splits_kernel<64, 0>);
    }
    BA_CUDA_TRY(cudaGetLastError());
    ctx->launches += 1;
  }
  return BA_OK;
}

// Ordering and binning: a stable LSD radix sort (digits of 4 to 11 bits, keys staged and ranked in shared
// memory, no inter-block waiting) and the kernels that turn its output into per-tile lists.
//
// (1) The Gaussians are sorted once by their 32-bit depth key (ties keep the index order: the sort is stable).
// (2) In that order every Gaussian emits one record per CELL of 4 x 4 tiles that its footprint reaches - the cell id
//     and a 16-bit mask of the tiles met inside the cell, as the preprocess left them - and the records are sorted by
//     cell id alone (a quarter of the elements and fewer bits than a sort of the (Gaussian, tile) instances).
// (3) A cell's records, still in depth order, are expanded into the lists of its 16 tiles: counts per chunk of 2048
//     records, one scan for the start of every tile and of every chunk inside it, then each chunk writes its
//     instances, the lanes that share a tile finding their slots with one ballot.
// The result is the instance list ordered by (tile, depth key, index), with its per-tile ranges.
#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kItems = 16;
constexpr int kSortTile = kSortThreads * kItems;   // 4096 elements per block iteration
constexpr int kMaxSortBlocks = 444;                // 3 resident CTAs x 148 SMs: one full wave
constexpr unsigned kFull = 0xffffffffu;
constexpr int kMaxDigitBits = 11;  // widest radix digit: 2048 bins
constexpr int kScanBlock = 256;   // Gaussians per block of the tiles-touched prefix sum and per CTA of the instance emission


// Block b sorts one contiguous range of the input, worked through in tiles of at most kSortTile elements.  While one
// tile per block is enough (count <= blocks x kSortTile) the ranges are equal, rounded up to a multiple of the block
// size, so that a full wave of CTAs shares the work evenly and every warp of a CTA ranks the same number of items.
// Beyond that, whole tiles are dealt out as evenly as they go: a pass costs a fixed latency per tile, and two full
// tiles in a few blocks measured faster than two half tiles in every block (0.40 against 0.45 ms per 8 views on
// 2 M records).  The grid is sized by the host's bound on the count; the ranges follow the count the kernels see
// (which may live on the device), so the work stays balanced either way.
constexpr int kMinPerBlock = 2048;
int sort_blocks(int64_t count) {
  const int64_t b = (count + kMinPerBlock - 1) / kMinPerBlock;
  return (int)(b < 1 ? 1 : b < kMaxSortBlocks ? b : kMaxSortBlocks);
}

struct BlockRange {
  int64_t begin, end;   // this block's elements
  int tiles, tile_len;  // worked through as `tiles` pieces of `tile_len` (the last one may be short)
};

__device__ __forceinline__ BlockRange block_range(int64_t count) {
  const int64_t nb = (int64_t)gridDim.x;
  BlockRange r;
  if (count <= nb * kSortTile) {
    int64_t per = (count + nb - 1) / nb;
    per = (per + kSortThreads - 1) / kSortThreads * kSortThreads;
    r.begin = min(count, (int64_t)blockIdx.x * per);
    r.end = min(count, r.begin + per);
    r.tiles = r.end > r.begin ? 1 : 0;
    r.tile_len = (int)per;
  } else {
    const int64_t tiles = (count + kSortTile - 1) / kSortTile;
    const int b = (int)blockIdx.x;
    const int each = (int)(tiles / nb), extra = (int)(tiles - (int64_t)each * nb);
    r.tiles = each + (b < extra ? 1 : 0);
    r.begin = ((int64_t)b * each + min(b, extra)) * kSortTile;
    r.end = min(count, r.begin + (int64_t)r.tiles * kSortTile);
    r.tile_len = kSortTile;
  }
  return r;
}

// Digit histogram of each block's contiguous range: table[digit][block] (digits of up to kMaxDigitBits bits).
__global__ void __launch_bounds__(kSortThreads) k_radix_hist(const uint32_t *__restrict__ keys, int64_t count,
                                                             const unsigned long long *__restrict__ count_dev,
                                                             int shift, int bits,
                                                             uint32_t *__restrict__ table, SortEpilogue ep) {
  dependency_wait();
  // the arrays the scatter of this pass accumulates into start from their neutral values
  if (ep.block_sums)
    for (int i = blockIdx.x * kSortThreads + threadIdx.x; i < ep.num_block_sums; i += gridDim.x * kSortThreads) ep.block_sums[i] = 0u;
  if (ep.ranges)
    for (int i = blockIdx.x * kSortThreads + threadIdx.x; i < 2 * ep.num_ranges; i += gridDim.x * kSortThreads)
      ep.ranges[i] = (i & 1) ? 0u : 0xffffffffu;
  if (count_dev) {
    const int64_t c = (int64_t)__ldg(count_dev);                    // the true length lives on the device
    if (ep.overflow && c > count && blockIdx.x == 0 && threadIdx.x == 0) *ep.overflow = 1u;   // lists were cut off: tell the host
    count = min(count, c);
  }
  // up to 256 digits: one histogram per warp (fewer collisions); more: two shared by the warps
  __shared__ uint32_t s_hist[2 << kMaxDigitBits];
  const int tid = threadIdx.x, warp = tid >> 5;
  const int nb = 1 << bits, copies = nb <= 256 ? kSortWarps : 2;
  const uint32_t mask = (uint32_t)nb - 1u;
  for (int k = tid; k < copies * nb; k += kSortThreads) s_hist[k] = 0;
  __syncthreads();
  const BlockRange r = block_range(count);
  uint32_t *mine = s_hist + (warp % copies) * nb;
  for (int64_t i = r.begin + tid; i < r.end; i += kSortThreads) atomicAdd(mine + ((__ldg(keys + i) >> shift) & mask), 1u);
  __syncthreads();
  for (int d = tid; d < nb; d += kSortThreads) {
    uint32_t t = 0;
    for (int w = 0; w < copies; ++w) t += s_hist[w * nb + d];
    table[(size_t)d * gridDim.x + blockIdx.x] = t;   // digit-major: one contiguous row per digit
  }
}

// Per digit (one CTA each): exclusive scan of the row of per-block counts, in place, and the row
// total.  Done once per pass here instead of by every scatter CTA.
__global__ void __launch_bounds__(256) k_radix_scan_rows(uint32_t *__restrict__ table, int nblocks,
                                                         uint32_t *__restrict__ totals) {
  dependency_wait();
  __shared__ uint32_t s_w[8];
  __shared__ uint32_t s_carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  uint32_t *row = table + (size_t)blockIdx.x * nblocks;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < nblocks; base += 256) {
    const int i = base + tid;
    const uint32_t v = i < nblocks ? row[i] : 0u;
    uint32_t inc = v;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const uint32_t t = __shfl_up_sync(0xffffffffu, inc, s);
      if (lane >= s) inc += t;
    }
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    uint32_t off = 0;
#pragma unroll
    for (int w = 0; w < 8; ++w) off += (w < warp) ? s_w[w] : 0u;
    const uint32_t carry = s_carry;
    if (i < nblocks) row[i] = carry + off + inc - v;
    __syncthreads();
    if (tid == 255) s_carry = carry + off + inc;
    __syncthreads();
  }
  if (tid == 0) totals[blockIdx.x] = s_carry;
}

// Exclusive prefix sums over kSortThreads * DPT values in thread-major order (thread t holds values t * DPT ..): each
// thread scans its own values, the thread totals are scanned across the block.
template <int DPT>
__device__ __forceinline__ void block_exclusive_scan(const uint32_t v[DPT], uint32_t out[DPT], uint32_t *s_warp_tot, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  uint32_t sum = 0;
#pragma unroll
  for (int j = 0; j < DPT; ++j) { out[j] = sum; sum += v[j]; }
  uint32_t inc = sum;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t t = __shfl_up_sync(kFull, inc, s);
    if (lane >= s) inc += t;
  }
  if (lane == 31) s_warp_tot[warp] = inc;
  __syncthreads();
  uint32_t off = inc - sum;
#pragma unroll
  for (int w = 0; w < kSortWarps; ++w) off += (w < warp) ? s_warp_tot[w] : 0u;
  __syncthreads();
#pragma unroll
  for (int j = 0; j < DPT; ++j) out[j] += off;
}

template <int BITS> constexpr size_t scatter_smem_bytes() {
  return sizeof(uint32_t) * (2 * kSortTile + (size_t)(kSortWarps + 2) * (BITS <= 8 ? 256 : (1 << BITS)) + kSortWarps);
}

// One pass: stable scatter of this block's range by the BITS-wide digit at `shift` (BITS up to kMaxDigitBits; the
// digit arrays hold max(256, 2^BITS) entries, thread t looking after digits t * DPT ..).  Slots past the
// end of the input carry the largest digit and sit at the end of the last tile, so they rank after
// every real key and are never written.
// EP selects the epilogue: 0 none, 1 block sums of a per-Gaussian count (last pass of the depth sort), 2 ranges of
// equal ids = key >> key_shift (last pass of the record sort: inside a block's run of one digit the keys are
// non-decreasing, because the earlier passes ordered the lower bits, so a change of id between neighbours of a run
// is a boundary; the two ends of a run may continue in another block and enter with an atomic min / max).
template <int BITS, int EP>
__global__ void __launch_bounds__(kSortThreads, BITS <= 9 ? 3 : 2) k_radix_scatter(
    const uint32_t *__restrict__ keys_in, const uint32_t *__restrict__ vals_in, uint32_t *__restrict__ keys_out,
    uint32_t *__restrict__ vals_out, int64_t count, const unsigned long long *__restrict__ count_dev, int shift,
    const uint32_t *__restrict__ table, const uint32_t *__restrict__ totals, int nblocks, SortEpilogue ep) {
  dependency_wait();
  constexpr int NB = BITS <= 8 ? 256 : (1 << BITS);   // entries of the digit arrays
  constexpr int DPT = NB / kSortThreads;              // digits per thread
  extern __shared__ __align__(16) uint32_t s_dyn[];
  uint32_t *s_keys = s_dyn, *s_vals = s_keys + kSortTile;
  uint32_t *s_warp_cnt = s_vals + kSortTile;          // [kSortWarps][NB]
  uint32_t *s_digit_start = s_warp_cnt + kSortWarps * NB, *s_base = s_digit_start + NB, *s_warp_tot = s_base + NB;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  if (count_dev) count = min(count, (int64_t)__ldg(count_dev));
  constexpr uint32_t kDigitMask = (1u << BITS) - 1u;

  // global base of every digit for this block: all smaller digits everywhere (scan of the row
  // totals) + the same digit in the blocks before this one (the row prefix from k_radix_scan_rows)
  {
    uint32_t tot[DPT], start[DPT];
#pragma unroll
    for (int j = 0; j < DPT; ++j) { const int d = tid * DPT + j; tot[j] = d <= (int)kDigitMask ? __ldg(totals + d) : 0u; }
    block_exclusive_scan<DPT>(tot, start, s_warp_tot, tid);
#pragma unroll
    for (int j = 0; j < DPT; ++j) {
      const int d = tid * DPT + j;
      s_base[d] = start[j] + (d <= (int)kDigitMask ? __ldg(table + (size_t)d * nblocks + blockIdx.x) : 0u);
    }
  }

  const BlockRange r = block_range(count);
  const int span = r.tile_len / kSortWarps;           // consecutive elements of a tile that one warp ranks
  const int items = span / 32;                        // ... as this many rows of 32 (at most kItems)
  for (int t = 0; t < r.tiles; ++t) {
    const int64_t tile_begin = r.begin + (int64_t)t * r.tile_len;
    if (tile_begin >= r.end) break;
    const int valid_count = (int)min((int64_t)r.tile_len, r.end - tile_begin);
    for (int k = tid; k < kSortWarps * NB; k += kSortThreads) s_warp_cnt[k] = 0;
    __syncthreads();
    uint32_t key[kItems], val[kItems];
    unsigned short rank[kItems];
    // all loads first (independent, in flight together), then the serial ranking chain
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int local = warp * span + it * 32 + lane;
      const bool ok = it < items && local < valid_count;
      const int64_t idx = tile_begin + local;
      key[it] = ok ? __ldg(keys_in + idx) : 0xffffffffu;
      val[it] = ok ? (vals_in ? __ldg(vals_in + idx) : (uint32_t)idx) : 0u;
    }
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      if (it >= items) break;                         // the same for every thread of the CTA
      const int local = warp * span + it * 32 + lane;
      const bool ok = local < valid_count;
      const uint32_t d = ok ? ((key[it] >> shift) & kDigitMask) : kDigitMask;
      // lanes with the same digit form a group; its first lane bumps the warp's counter once and
      // hands the old value to the group.  A warp's shared-memory atomics execute in program order,
      // so the 16 items need no barrier between them and their latencies overlap.
      // The group comes from one ballot per digit bit: a fixed cost, where the match instruction
      // takes time in proportion to the number of different digits in the warp.
      uint32_t peers = kFull;
#pragma unroll
      for (int b = 0; b < BITS; ++b) {
        const bool bit = (d >> b) & 1u;
        const uint32_t m = __ballot_sync(kFull, bit);
        peers &= bit ? m : ~m;
      }
      const int leader = __ffs(peers) - 1;
      uint32_t prior = 0;
      if (lane == leader) prior = atomicAdd(&s_warp_cnt[warp * NB + d], (uint32_t)__popc(peers));
      prior = __shfl_sync(kFull, prior, leader);
      rank[it] = (unsigned short)(prior + __popc(peers & lt_mask));
    }
    __syncthreads();
    // per digit: exclusive scan over warps, then over digits
    uint32_t cnt[DPT], dstart[DPT];
#pragma unroll
    for (int j = 0; j < DPT; ++j) {
      const int d = tid * DPT + j;
      uint32_t c = 0;
#pragma unroll
      for (int w = 0; w < kSortWarps; ++w) {
        const uint32_t x = s_warp_cnt[w * NB + d];
        s_warp_cnt[w * NB + d] = c;
        c += x;
      }
      cnt[j] = c;
    }
    block_exclusive_scan<DPT>(cnt, dstart, s_warp_tot, tid);
#pragma unroll
    for (int j = 0; j < DPT; ++j) s_digit_start[tid * DPT + j] = dstart[j];
    __syncthreads();
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      if (it >= items) break;
      const int local = warp * span + it * 32 + lane;
      const uint32_t d = (local < valid_count) ? ((key[it] >> shift) & kDigitMask) : kDigitMask;
      const uint32_t pos = s_digit_start[d] + s_warp_cnt[warp * NB + d] + rank[it];
      s_keys[pos] = key[it];
      s_vals[pos] = val[it];
    }
    __syncthreads();
    for (int j0 = 0; j0 < valid_count; j0 += kSortThreads) {
      const int j = j0 + tid;
      const bool ok = j < valid_count;
      uint32_t k = 0, d = 0, gpos = 0, v = 0;
      if (ok) {
        k = s_keys[j];
        d = (k >> shift) & kDigitMask;
        gpos = s_base[d] + ((uint32_t)j - s_digit_start[d]);
        v = s_vals[j];
        keys_out[gpos] = k;
        vals_out[gpos] = v;
      }
      if (EP == 1) {
        // the Gaussian's count, added to the sum of its block of kScanBlock sorted positions; a warp whose
        // lanes all fall into one block (the usual case: a run is contiguous) adds once
        uint32_t tt = ok ? (__ldg(ep.counts + v) & ep.count_mask) : 0u;
        const uint32_t blk = gpos / kScanBlock, blk0 = __shfl_sync(kFull, blk, 0);
        if (__all_sync(kFull, !ok || blk == blk0)) {
#pragma unroll
          for (int sft = 16; sft > 0; sft >>= 1) tt += __shfl_xor_sync(kFull, tt, sft);
          if (lane == 0 && tt) atomicAdd(ep.block_sums + blk0, tt);
        } else if (tt) {
          atomicAdd(ep.block_sums + blk, tt);
        }
      }
      if (EP == 2 && ok) {
        const uint32_t run_first = s_digit_start[d];
        const uint32_t run_end = d == kDigitMask ? (uint32_t)valid_count : s_digit_start[d + 1];   // slots past the input hold no run
        const uint32_t id = k >> ep.key_shift;
        if ((uint32_t)j == run_first) atomicMin(ep.ranges + 2 * id, gpos);
        else if ((s_keys[j - 1] >> ep.key_shift) != id) ep.ranges[2 * id] = gpos;
        if ((uint32_t)j + 1 == run_end) atomicMax(ep.ranges + 2 * id + 1, gpos + 1);
        else if ((s_keys[j + 1] >> ep.key_shift) != id) ep.ranges[2 * id + 1] = gpos + 1;
      }
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < DPT; ++j) s_base[tid * DPT + j] += cnt[j];
    __syncthreads();
  }
}

__global__ void k_flag_if_greater(const unsigned long long *__restrict__ value, unsigned long long bound, uint32_t *__restrict__ flag) {
  if (*value > bound) *flag = 1u;
}

__global__ void k_iota(uint32_t *__restrict__ out, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = (uint32_t)i;
}

// ---- cell records in depth order ---------------------------------------------------------------
// Every Gaussian, in depth order, writes its records (cell id << 16 | tile mask) and its id.  A Gaussian of at most
// 3 x 3 cells copies what the preprocess stored; a larger one is worked out again by its whole warp: per row of cells
// four lanes take the four tile rows, then the lanes take one cell each.
__global__ void __launch_bounds__(kScanBlock) k_emit_records(
    const uint32_t *__restrict__ order, const uint32_t *__restrict__ cell_count, const uint32_t *__restrict__ cell_records,
    const uint16_t *__restrict__ rect, const float *__restrict__ mean2d, const float *__restrict__ conic_opacity,
    const uint32_t *__restrict__ block_sums, int64_t n, int cgx, int W, int H, uint32_t capacity,
    uint32_t *__restrict__ rec_keys, uint32_t *__restrict__ rec_vals, unsigned long long *__restrict__ rec_total,
    uint32_t *__restrict__ overflow) {
  dependency_wait();
  __shared__ uint32_t s_w[kScanBlock / 32], s_before[kScanBlock / 32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t i = (int64_t)blockIdx.x * kScanBlock + tid;
  uint32_t g = 0, cc = 0;
  if (i < n) {
    g = __ldg(order + i);
    cc = __ldg(cell_count + g);
  }
  const uint32_t cnt = cc & ~kCellBig;
  uint32_t inc = cnt;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t t = __shfl_up_sync(kFull, inc, s);
    if (lane >= s) inc += t;
  }
  if (lane == 31) s_w[warp] = inc;
  // records of all CTAs before this one: the sums per kScanBlock Gaussians come from the last pass of the depth
  // sort; every CTA adds up its own prefix (a few loads per thread) instead of a scan kernel doing it for all
  uint32_t before = 0;
  for (int k = tid; k < (int)blockIdx.x; k += kScanBlock) before += __ldg(block_sums + k);
#pragma unroll
  for (int sft = 16; sft > 0; sft >>= 1) before += __shfl_xor_sync(kFull, before, sft);
  if (lane == 0) s_before[warp] = before;
  __syncthreads();
  uint32_t off = 0;
#pragma unroll
  for (int k = 0; k < kScanBlock / 32; ++k) off += s_before[k] + ((k < warp) ? s_w[k] : 0u);
  off += inc - cnt;
  if (blockIdx.x == gridDim.x - 1 && tid == kScanBlock - 1) {   // the last thread of all: its end is the number of records
    *rec_total = (unsigned long long)off + cnt;
    if (off + cnt > capacity) *overflow = 1u;                    // more records than the buffers hold: tell the host
  }
  if (cnt && !(cc & kCellBig)) {
    const uint32_t *src = cell_records + (size_t)g * kCellSlots;
    for (uint32_t k = 0; k < cnt; ++k) {
      if (off + k < capacity) {   // never past the buffers, even if the count was taken on the device
        rec_keys[off + k] = __ldg(src + k);
        rec_vals[off + k] = g;
      }
    }
  }
  uint32_t big = __ballot_sync(kFull, (cc & kCellBig) != 0u);
  while (big) {
    const int src = __ffs(big) - 1;
    big &= big - 1;
    const uint32_t s_g = __shfl_sync(kFull, g, src);
    uint32_t p = __shfl_sync(kFull, off, src);
    // the owner's projected values reach every lane by a broadcast load
    const ushort4 r = __ldg(reinterpret_cast<const ushort4 *>(rect) + s_g);
    const float2 m = __ldg(reinterpret_cast<const float2 *>(mean2d) + s_g);
    const float4 q = __ldg(reinterpret_cast<const float4 *>(conic_opacity) + s_g);
    TileSpans sp;
    sp.setup(m.x, m.y, q.x, q.y, q.z, footprint_tau(q.w), W, H);
    const int cy0 = r.y >> 2, cy1 = ((int)r.w - 1) >> 2;
    for (int cy = cy0; cy <= cy1; ++cy) {
      // lanes 0..3: the tile rows of this row of cells
      int xa = 0, xb = 0;
      const int ty = 4 * cy + lane;
      const bool has = lane < 4 && ty >= (int)r.y && ty < (int)r.w && sp.row(ty, r.x, r.z, xa, xb);
      int lo = has ? (xa >> 2) : (1 << 30), hi = has ? ((xb - 1) >> 2) : -1;
      lo = min(lo, __shfl_xor_sync(kFull, lo, 1)); hi = max(hi, __shfl_xor_sync(kFull, hi, 1));
      lo = min(lo, __shfl_xor_sync(kFull, lo, 2)); hi = max(hi, __shfl_xor_sync(kFull, hi, 2));
      lo = __shfl_sync(kFull, lo, 0); hi = __shfl_sync(kFull, hi, 0);
      if (hi < lo) continue;
      int ra[4], rb[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        ra[k] = __shfl_sync(kFull, has ? xa : 0, k);
        rb[k] = __shfl_sync(kFull, has ? xb : 0, k);
      }
      for (int cb = lo; cb <= hi; cb += 32) {
        const int cx = cb + lane;
        if (cx <= hi) {
          uint32_t mask = 0u;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const int a0 = max(ra[k], 4 * cx) - 4 * cx, b0 = min(rb[k], 4 * cx + 4) - 4 * cx;
            if (b0 > a0) mask |= (((1u << (b0 - a0)) - 1u) << a0) << (4 * k);
          }
          const uint32_t dst = p + (uint32_t)(cx - lo);
          if (dst < capacity) {
            rec_keys[dst] = ((uint32_t)(cy * cgx + cx) << 16) | mask;
            rec_vals[dst] = s_g;
          }
        }
      }
      p += (uint32_t)(hi - lo + 1);
    }
  }
}

// ---- from the sorted records of a cell to the lists of its tiles ----------------------------------
// Chunks: the records of cell c, [range_c.start, range_c.end), in pieces of kCellChunk; chunk_first[c] = number of
// chunks of the cells before c.  A cell without records comes in as (0xffffffff, 0), the neutral values of the
// range epilogue.
__global__ void __launch_bounds__(1024) k_cell_chunks(const uint32_t *__restrict__ cell_ranges, int num_cells,
                                                      uint32_t *__restrict__ chunk_first) {
  dependency_wait();
  __shared__ uint32_t s_w[32];
  __shared__ uint32_t s_carry;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_carry = 0;
  __syncthreads();
  for (int base = 0; base < num_cells; base += 1024) {
    const int c = base + tid;
    uint32_t v = 0;
    if (c < num_cells) {
      const uint32_t s0 = cell_ranges[2 * c], e0 = cell_ranges[2 * c + 1];
      v = e0 > s0 ? (e0 - s0 + kCellChunk - 1) / kCellChunk : 0u;
    }
    uint32_t inc = v;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const uint32_t t = __shfl_up_sync(kFull, inc, s);
      if (lane >= s) inc += t;
    }
    if (lane == 31) s_w[warp] = inc;
    __syncthreads();
    if (warp == 0) {
      uint32_t w = s_w[lane], winc = w;
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const uint32_t t = __shfl_up_sync(kFull, winc, s);
        if (lane >= s) winc += t;
      }
      s_w[lane] = winc - w;
    }
    __syncthreads();
    const uint32_t carry = s_carry;
    if (c < num_cells) chunk_first[c] = carry + s_w[warp] + inc - v;
    __syncthreads();
    if (tid == 1023) s_carry = carry + s_w[warp] + inc;
    __syncthreads();
  }
  if (tid == 0) chunk_first[num_cells] = s_carry;
}

// The cell and the record range of chunk q, or false if there is no such chunk.
__device__ __forceinline__ bool chunk_of(uint32_t q, const uint32_t *__restrict__ chunk_first, const uint32_t *__restrict__ cell_ranges,
                                         int num_cells, int &cell, uint32_t &begin, uint32_t &end) {
  if (q >= __ldg(chunk_first + num_cells)) return false;
  int lo = 0, hi = num_cells - 1;     // largest c with chunk_first[c] <= q (cells without records share a value: take the last)
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (__ldg(chunk_first + mid) <= q) lo = mid; else hi = mid - 1;
  }
  cell = lo;
  const uint32_t s0 = __ldg(cell_ranges + 2 * lo), e0 = __ldg(cell_ranges + 2 * lo + 1);
  begin = s0 + (q - __ldg(chunk_first + lo)) * kCellChunk;
  end = min(begin + (uint32_t)kCellChunk, e0);
  return true;
}

// The 16 tile counts of the records a lane holds (masks of up to 8 records), as four words of four byte counters:
// one multiplication spreads the four bits of a tile row of the cell over the four bytes of a word.
__device__ __forceinline__ void count_masks(const uint32_t mask[8], int have, uint32_t acc[4]) {
  acc[0] = acc[1] = acc[2] = acc[3] = 0u;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t m = k < have ? mask[k] : 0u;
#pragma unroll
    for (int r = 0; r < 4; ++r) acc[r] += (((m >> (4 * r)) & 15u) * 0x00204081u) & 0x01010101u;
  }
}

// Sum over the warp of the byte counters, widened to 16 bits on the way (8 records x 32 lanes = 256 at most): tile
// 4 r + b of the cell ends in bits [16 (b & 1), +16) of word r * 2 + (b >> 1), in every lane.
__device__ __forceinline__ void warp_sum_counts(const uint32_t acc[4], uint32_t out[8]) {
#pragma unroll
  for (int r = 0; r < 4; ++r) {
    out[2 * r] = (acc[r] & 0xffu) | ((acc[r] & 0xff00u) << 8);
    out[2 * r + 1] = ((acc[r] >> 16) & 0xffu) | ((acc[r] >> 8) & 0xff0000u);
  }
#pragma unroll
  for (int w = 0; w < 8; ++w)
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) out[w] += __shfl_xor_sync(kFull, out[w], s);
}
__device__ __forceinline__ uint32_t tile_count_of(const uint32_t sums[8], int t) {   // t = 4 r + b
  return (sums[2 * (t >> 2) + ((t & 3) >> 1)] >> (16 * (t & 1))) & 0xffffu;
}

constexpr int kExpandThreads = 256;
constexpr int kExpandWarps = kExpandThreads / 32;

// Per chunk: how many instances it holds for each of the 16 tiles of its cell.
__global__ void __launch_bounds__(kExpandThreads) k_chunk_counts(const uint32_t *__restrict__ rec_keys,
                                                                 const uint32_t *__restrict__ cell_ranges,
                                                                 const uint32_t *__restrict__ chunk_first, int num_cells,
                                                                 uint32_t *__restrict__ chunk_counts) {
  dependency_wait();
  __shared__ uint32_t s_cnt[kExpandWarps][16];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int cell;
  uint32_t begin, end;
  if (!chunk_of(blockIdx.x, chunk_first, cell_ranges, num_cells, cell, begin, end)) return;
  // warp w holds records [begin + 256 w, + 256): lane l the records 256 w + 32 k + l, k = 0..7
  uint32_t mask[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t idx = begin + (uint32_t)(256 * warp + 32 * k + lane);
    mask[k] = idx < end ? (__ldg(rec_keys + idx) & 0xffffu) : 0u;
  }
  uint32_t acc[4], sums[8];
  count_masks(mask, 8, acc);
  warp_sum_counts(acc, sums);
  if (lane < 16) s_cnt[warp][lane] = tile_count_of(sums, lane);
  __syncthreads();
  if (tid < 16) {
    uint32_t t = 0;
#pragma unroll
    for (int w = 0; w < kExpandWarps; ++w) t += s_cnt[w][tid];
    chunk_counts[(size_t)blockIdx.x * 16 + tid] = t;
  }
}

// Per cell (one warp each, lanes 0..15 = its tiles): where each chunk's instances of a tile begin inside the tile's
// list (the running sum of the chunks' counts, in chunk order) and the length of that list.
__global__ void __launch_bounds__(256) k_cell_prefix(const uint32_t *__restrict__ chunk_first, const uint32_t *__restrict__ chunk_counts,
                                                     int gx, int gy, int cgx, int num_cells, uint32_t *__restrict__ chunk_bases,
                                                     uint32_t *__restrict__ tile_counts) {
  dependency_wait();
  const int lane = threadIdx.x & 31, cell = blockIdx.x * 8 + (threadIdx.x >> 5);
  if (cell >= num_cells || lane >= 16) return;
  const uint32_t q0 = __ldg(chunk_first + cell), q1 = __ldg(chunk_first + cell + 1);
  uint32_t run = 0;
  uint32_t q = q0;
  for (; q + 4 <= q1; q += 4) {   // four independent loads in flight
    const uint32_t v0 = __ldg(chunk_counts + (size_t)q * 16 + lane), v1 = __ldg(chunk_counts + (size_t)(q + 1) * 16 + lane);
    const uint32_t v2 = __ldg(chunk_counts + (size_t)(q + 2) * 16 + lane), v3 = __ldg(chunk_counts + (size_t)(q + 3) * 16 + lane);
    chunk_bases[(size_t)q * 16 + lane] = run; run += v0;
    chunk_bases[(size_t)(q + 1) * 16 + lane] = run; run += v1;
    chunk_bases[(size_t)(q + 2) * 16 + lane] = run; run += v2;
    chunk_bases[(size_t)(q + 3) * 16 + lane] = run; run += v3;
  }
  for (; q < q1; ++q) {
    chunk_bases[(size_t)q * 16 + lane] = run;
    run += __ldg(chunk_counts + (size_t)q * 16 + lane);
  }
  const int tx = 4 * (cell % cgx) + (lane & 3), ty = 4 * (cell / cgx) + (lane >> 2);
  if (tx < gx && ty < gy) tile_counts[ty * gx + tx] = run;
}

// One CTA: the exclusive scan of the tile counts in tile order = the tile ranges, and the launch order of the blend
// CTAs (tiles by decreasing list length in log2 buckets: the long tiles start first and the short ones fill the tail;
// the order inside a bucket is whatever the atomics give, it affects scheduling only, never a result).
__global__ void __launch_bounds__(1024) k_tile_scan(const uint32_t *__restrict__ tile_counts, int num_tiles, uint32_t capacity,
                                                    uint32_t *__restrict__ tile_starts, uint32_t *__restrict__ ranges,
                                                    uint32_t *__restrict__ order) {
  dependency_wait();
  __shared__ uint32_t s_w[32];
  __shared__ uint32_t s_cnt[33], s_off[33];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid < 33) s_cnt[tid] = 0;
  __syncthreads();
  // thread t takes the tiles [t per, (t + 1) per): one pass over its counts, one scan of the thread sums
  const int per = (num_tiles + 1023) / 1024, first = tid * per, last = min(first + per, num_tiles);
  uint32_t sum = 0;
  for (int t = first; t < last; ++t) {
    const uint32_t v = tile_counts[t];
    sum += v;
    atomicAdd(&s_cnt[v ? 32 - __clz(v) : 0], 1u);
  }
  uint32_t inc = sum;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t u = __shfl_up_sync(kFull, inc, s);
    if (lane >= s) inc += u;
  }
  if (lane == 31) s_w[warp] = inc;
  __syncthreads();
  if (warp == 0) {
    uint32_t w = s_w[lane], winc = w;
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const uint32_t u = __shfl_up_sync(kFull, winc, s);
      if (lane >= s) winc += u;
    }
    s_w[lane] = winc - w;
  }
  if (tid == 0) {
    uint32_t off = 0;
    for (int b = 32; b >= 0; --b) { s_off[b] = off; off += s_cnt[b]; }
  }
  __syncthreads();
  uint32_t start = s_w[warp] + inc - sum;
  for (int t = first; t < last; ++t) {
    const uint32_t v = tile_counts[t];
    tile_starts[t] = start;
    // a tile without instances: (0, 0); never past the capacity of the instance buffers (a device-side count may
    // exceed it: the lists are then cut off and the host is told)
    const uint32_t s0 = min(start, capacity), e0 = start + v < start ? capacity : min(start + v, capacity);
    ranges[2 * t] = e0 > s0 ? s0 : 0u;
    ranges[2 * t + 1] = e0 > s0 ? e0 : 0u;
    order[atomicAdd(&s_off[v ? 32 - __clz(v) : 0], 1u)] = (uint32_t)t;
    start += v;
  }
}

__device__ __forceinline__ void store_if(bool p, uint32_t *addr, uint32_t v) {
  asm volatile("{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %0, 0;\n\t@q st.global.u32 [%1], %2;\n\t}" :: "r"((uint32_t)p), "l"(addr), "r"(v) : "memory");
}

// Per chunk: write its instances.  A warp's records are consecutive in depth order, 32 at a time.  A record's slot
// in the list of tile t is the tile's running position plus the number of lower lanes that also list t: the 16
// indicator bits of a lane's mask are spread over four words of byte counters and one warp-wide prefix sum of those
// four words ranks all 16 tiles at once (at most 32 per byte).  The running positions start from the tile's range,
// the chunk's offset inside it and what the warps before this one hold; every lane keeps all 16 of them.
__global__ void __launch_bounds__(kExpandThreads) k_expand(const uint32_t *__restrict__ rec_keys, const uint32_t *__restrict__ rec_vals,
                                                           const uint32_t *__restrict__ cell_ranges,
                                                           const uint32_t *__restrict__ chunk_first, int num_cells,
                                                           const uint32_t *__restrict__ chunk_bases,
                                                           const uint32_t *__restrict__ tile_starts, int gx, int gy, int cgx,
                                                           uint32_t capacity, uint32_t *__restrict__ out_vals) {
  dependency_wait();
  __shared__ uint32_t s_cnt[kExpandWarps][16];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  int cell;
  uint32_t begin, end;
  if (!chunk_of(blockIdx.x, chunk_first, cell_ranges, num_cells, cell, begin, end)) return;
  uint32_t mask[8], gid[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t idx = begin + (uint32_t)(256 * warp + 32 * k + lane);
    const bool ok = idx < end;
    mask[k] = ok ? (__ldg(rec_keys + idx) & 0xffffu) : 0u;
    gid[k] = ok ? __ldg(rec_vals + idx) : 0u;
  }
  uint32_t acc[4], sums[8];
  count_masks(mask, 8, acc);
  warp_sum_counts(acc, sums);
  if (lane < 16) s_cnt[warp][lane] = tile_count_of(sums, lane);
  __syncthreads();
  // lane t < 16 works out where tile t of the cell continues, then every lane takes a copy of all 16
  const int tx0 = 4 * (cell % cgx), ty0 = 4 * (cell / cgx);
  uint32_t mine = 0;
  if (lane < 16) {
    const int tx = tx0 + (lane & 3), ty = ty0 + (lane >> 2);
    if (tx < gx && ty < gy) {   // (a tile of the cell outside the image has no instances)
      mine = __ldg(tile_starts + ty * gx + tx) + __ldg(chunk_bases + (size_t)blockIdx.x * 16 + lane);
      for (int w = 0; w < warp; ++w) mine += s_cnt[w][lane];
    }
  }
  uint32_t cur[16];
#pragma unroll
  for (int t = 0; t < 16; ++t) cur[t] = __shfl_sync(kFull, mine, t);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint32_t m = mask[k];
    if (__ballot_sync(kFull, m != 0u) == 0u) continue;
    uint32_t incl[4], own[4], tot[4];
#pragma unroll
    for (int r = 0; r < 4; ++r) {
      own[r] = (((m >> (4 * r)) & 15u) * 0x00204081u) & 0x01010101u;
      incl[r] = own[r];
    }
#pragma unroll
    for (int sft = 1; sft < 32; sft <<= 1) {
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const uint32_t u = __shfl_up_sync(kFull, incl[r], sft);
        if (lane >= sft) incl[r] += u;
      }
    }
#pragma unroll
    for (int r = 0; r < 4; ++r) tot[r] = __shfl_sync(kFull, incl[r], 31);
#pragma unroll
    for (int t = 0; t < 16; ++t) {
      const int r = t >> 2, sh = 8 * (t & 3);
      // one predicated store (no branch): the lane lists tile t and the slot lies inside the buffer
      const uint32_t pos = cur[t] + (((incl[r] - own[r]) >> sh) & 0xffu);
      store_if(((m >> t) & 1u) != 0u && pos < capacity, out_vals + pos, gid[k]);
      cur[t] += (tot[r] >> sh) & 0xffu;
    }
  }
}

}  // namespace

size_t sort_scratch_bytes(int64_t count) { return ((size_t)sort_blocks(count) + 1) * (1 << kMaxDigitBits) * sizeof(uint32_t); }

namespace {
template <int BITS, int EP>
void launch_scatter(int blocks, const uint32_t *src_k, const uint32_t *src_v, uint32_t *dst_k, uint32_t *dst_v, int64_t count,
                    const unsigned long long *count_dev, int shift, const uint32_t *table, const uint32_t *totals,
                    const SortEpilogue &ep, cudaStream_t st) {
  constexpr size_t smem = scatter_smem_bytes<BITS>();
  static bool opted[64] = {};
  int dev = 0;
  cudaGetDevice(&dev);
  if (smem > 48 * 1024 && dev >= 0 && dev < 64 && !opted[dev]) {
    cudaFuncSetAttribute(k_radix_scatter<BITS, EP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    opted[dev] = true;
  }
  launch_chained(k_radix_scatter<BITS, EP>, blocks, kSortThreads, smem, st, src_k, src_v, dst_k, dst_v, count, count_dev, shift, table,
                 totals, blocks, ep);
}
}  // namespace

int launch_radix_sort(const uint32_t *keys_in, const uint32_t *vals_in, uint32_t *keys_out, uint32_t *vals_out,
                       uint32_t *tmp_keys, uint32_t *tmp_vals, int64_t count, const unsigned long long *count_dev,
                       int first_bit, int num_bits, int max_digit_bits, void *scratch, const SortEpilogue *epilogue,
                       cudaStream_t st) {
  if (count <= 0) return 0;
  const int blocks = sort_blocks(count);
  const int passes = radix_passes(num_bits, max_digit_bits);
  int bits = (num_bits + passes - 1) / passes;     // digits of equal width: 13 bits sort as 7 + 6 under a limit of 8
  if (bits < 4) bits = 4;                          // (bits above the keys' range are zero: sorting on them changes nothing)
  uint32_t *table = static_cast<uint32_t *>(scratch);
  uint32_t *totals = table + ((size_t)blocks << bits);
  const uint32_t *src_k = keys_in, *src_v = vals_in;
  const SortEpilogue none = {nullptr, 0u, nullptr, 0, nullptr, 0, 0, nullptr};
  for (int p = 0; p < passes; ++p) {
    const bool to_out = ((passes - 1 - p) % 2) == 0;
    uint32_t *dst_k = to_out ? keys_out : tmp_keys, *dst_v = to_out ? vals_out : tmp_vals;
    const SortEpilogue ep = (p == passes - 1 && epilogue) ? *epilogue : none;
    const int mode = ep.block_sums ? 1 : ep.ranges ? 2 : 0;
    const int shift = first_bit + bits * p;
    launch_chained(k_radix_hist, blocks, kSortThreads, 0, st, src_k, count, count_dev, shift, bits, table, ep);
    launch_chained(k_radix_scan_rows, 1 << bits, 256, 0, st, table, blocks, totals);
#define GS_ARGS blocks, src_k, src_v, dst_k, dst_v, count, count_dev, shift, table, totals, ep, st
#define GS_SCATTER(B)                                             \
  case B:                                                         \
    if (mode == 2) launch_scatter<B, 2>(GS_ARGS);                 \
    else launch_scatter<B, 0>(GS_ARGS);                           \
    break;
    switch (bits) {
      GS_SCATTER(4) GS_SCATTER(5) GS_SCATTER(6) GS_SCATTER(7) GS_SCATTER(9) GS_SCATTER(10)
      case 8:
        if (mode == 1) launch_scatter<8, 1>(GS_ARGS);
        else if (mode == 2) launch_scatter<8, 2>(GS_ARGS);
        else launch_scatter<8, 0>(GS_ARGS);
        break;
      default:
        if (mode == 2) launch_scatter<11, 2>(GS_ARGS);
        else launch_scatter<11, 0>(GS_ARGS);
    }
#undef GS_SCATTER
#undef GS_ARGS
    src_k = dst_k;
    src_v = dst_v;
  }
  return 3 * passes;
}

int radix_passes(int num_bits, int max_digit_bits) {
  const int m = max_digit_bits < 4 ? 4 : max_digit_bits > kMaxDigitBits ? kMaxDigitBits : max_digit_bits;
  const int p = (num_bits + m - 1) / m;
  return p < 1 ? 1 : p;
}

size_t scan_scratch_bytes(int64_t n) { return (size_t)((n + kScanBlock - 1) / kScanBlock + 1) * sizeof(uint32_t); }
int num_scan_blocks(int64_t n) { return (int)((n + kScanBlock - 1) / kScanBlock); }

int launch_emit_records(const uint32_t *depth_order, const uint32_t *cell_count, const uint32_t *cell_records,
                        const uint16_t *rect, const float *mean2d, const float *conic_opacity, const uint32_t *block_sums,
                        uint32_t *rec_keys, uint32_t *rec_vals, unsigned long long *rec_total, uint32_t *overflow, int64_t n,
                        int cgx, int W, int H, int64_t capacity, cudaStream_t st) {
  if (n <= 0) return 0;
  const uint32_t cap = capacity > 0xffffffffll ? 0xffffffffu : (uint32_t)capacity;
  launch_chained(k_emit_records, num_scan_blocks(n), kScanBlock, 0, st, depth_order, cell_count, cell_records, rect, mean2d, conic_opacity,
                 block_sums, n, cgx, W, H, cap, rec_keys, rec_vals, rec_total, overflow);
  return 1;
}

int max_chunks(int64_t record_capacity, int num_cells) { return (int)((record_capacity + kCellChunk - 1) / kCellChunk) + num_cells; }

int launch_expand(const uint32_t *rec_keys, const uint32_t *rec_vals, const uint32_t *cell_ranges, const CellScratch &cs,
                  int64_t record_capacity, int64_t pair_capacity, int gx, int gy, int cgx, int cgy,
                  uint32_t *sorted_vals, uint32_t *tile_ranges, uint32_t *tile_order, cudaStream_t st) {
  const int num_cells = cgx * cgy, chunks = max_chunks(record_capacity, num_cells);
  const uint32_t cap = pair_capacity > 0xffffffffll ? 0xffffffffu : (uint32_t)pair_capacity;
  launch_chained(k_cell_chunks, 1, 1024, 0, st, cell_ranges, num_cells, cs.chunk_first);
  launch_chained(k_chunk_counts, chunks, kExpandThreads, 0, st, rec_keys, cell_ranges, cs.chunk_first, num_cells, cs.chunk_counts);
  launch_chained(k_cell_prefix, (num_cells + 7) / 8, 256, 0, st, cs.chunk_first, cs.chunk_counts, gx, gy, cgx, num_cells, cs.chunk_bases,
                 cs.tile_counts);
  launch_chained(k_tile_scan, 1, 1024, 0, st, cs.tile_counts, gx * gy, cap, cs.tile_starts, tile_ranges, tile_order);
  launch_chained(k_expand, chunks, kExpandThreads, 0, st, rec_keys, rec_vals, cell_ranges, cs.chunk_first, num_cells, cs.chunk_bases,
                 cs.tile_starts, gx, gy, cgx, cap, sorted_vals);
  return 5;
}

void launch_flag_if_greater(const unsigned long long *value, unsigned long long bound, uint32_t *flag, cudaStream_t st) {
  k_flag_if_greater<<<1, 1, 0, st>>>(value, bound, flag);
}

// No record was sorted (no Gaussian, or none that reaches a tile): every tile is empty.
int launch_empty_binning(uint32_t *tile_ranges, uint32_t *tile_order, int num_tiles, cudaStream_t st) {
  cudaMemsetAsync(tile_ranges, 0, (size_t)num_tiles * 2 * sizeof(uint32_t), st);
  k_iota<<<(num_tiles + 255) / 256, 256, 0, st>>>(tile_order, num_tiles);
  return 1;
}

}  // namespace gs

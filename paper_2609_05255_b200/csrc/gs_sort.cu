// Ordering and binning: a stable LSD radix sort (digits of up to 8 bits, keys staged and ranked in shared
// memory, no inter-block waiting), the prefix sum of tiles touched in depth order, instance
// generation and per-tile ranges.
//
// Two-stage ordering: (1) the Gaussians are sorted once by their 32-bit depth key (ties keep the
// index order because the sort is stable); (2) instances are emitted in that order and sorted by
// tile id only (ceil(log2(tiles)) bits).  The result is the order by (tile, depth key, index).
#include "gs_device.cuh"

namespace gs {
namespace {

constexpr int kSortThreads = 256;
constexpr int kSortWarps = kSortThreads / 32;
constexpr int kItems = 16;
constexpr int kSortTile = kSortThreads * kItems;   // 4096 elements per block iteration
constexpr int kMaxSortBlocks = 444;                // 3 resident CTAs x 148 SMs: one full wave
constexpr unsigned kFull = 0xffffffffu;
constexpr int kScanBlock = 256;   // Gaussians per block of the tiles-touched prefix sum and per CTA of the instance emission

// Block b sorts tiles_per_block (+ 1 if b < extra) consecutive tiles of kSortTile elements: the tiles are dealt
// out as evenly as whole tiles allow over one full wave of CTAs.
struct SortPlan { int blocks; int tiles_per_block; int extra; };

SortPlan plan_for(int64_t count) {
  const int64_t tiles = (count + kSortTile - 1) / kSortTile;
  SortPlan p;
  p.blocks = (int)(tiles < kMaxSortBlocks ? tiles : kMaxSortBlocks);
  if (p.blocks < 1) p.blocks = 1;
  p.tiles_per_block = (int)(tiles / p.blocks);
  p.extra = (int)(tiles - (int64_t)p.tiles_per_block * p.blocks);
  return p;
}

// First tile and number of tiles of a block under the plan.
__device__ __forceinline__ void block_tiles(int tiles_per_block, int extra, int64_t &first, int &num) {
  const int b = (int)blockIdx.x;
  first = (int64_t)b * tiles_per_block + min(b, extra);
  num = tiles_per_block + (b < extra ? 1 : 0);
}

// Digit histogram of each block's contiguous range: table[block][digit].
__global__ void __launch_bounds__(kSortThreads) k_radix_hist(const uint32_t *__restrict__ keys, int64_t count,
                                                             const unsigned long long *__restrict__ count_dev,
                                                             int shift, uint32_t mask, int tiles_per_block, int extra,
                                                             uint32_t *__restrict__ table, SortEpilogue ep) {
  // the arrays the scatter of this pass accumulates into start from their neutral values
  if (ep.block_sums)
    for (int i = blockIdx.x * kSortThreads + threadIdx.x; i < ep.num_block_sums; i += gridDim.x * kSortThreads) ep.block_sums[i] = 0u;
  if (ep.ranges)
    for (int i = blockIdx.x * kSortThreads + threadIdx.x; i < 2 * ep.num_tiles; i += gridDim.x * kSortThreads)
      ep.ranges[i] = (i & 1) ? 0u : 0xffffffffu;
  if (count_dev) {
    const int64_t c = (int64_t)__ldg(count_dev);                    // the true length lives on the device
    if (ep.overflow && c > count && blockIdx.x == 0 && threadIdx.x == 0) *ep.overflow = 1u;   // lists were cut off: tell the host
    count = min(count, c);
  }
  __shared__ uint32_t s_hist[kSortWarps][256];
  const int tid = threadIdx.x, warp = tid >> 5;
  for (int k = tid; k < kSortWarps * 256; k += kSortThreads) (&s_hist[0][0])[k] = 0;
  __syncthreads();
  int64_t first_tile;
  int my_tiles;
  block_tiles(tiles_per_block, extra, first_tile, my_tiles);
  const int64_t begin = first_tile * kSortTile;
  int64_t end = begin + (int64_t)my_tiles * kSortTile;
  if (end > count) end = count;
  for (int64_t i = begin + tid; i < end; i += kSortThreads) {
    const uint32_t d = (__ldg(keys + i) >> shift) & mask;
    atomicAdd(&s_hist[warp][d], 1u);
  }
  __syncthreads();
  uint32_t s = 0;
#pragma unroll
  for (int w = 0; w < kSortWarps; ++w) s += s_hist[w][tid];
  table[(size_t)tid * gridDim.x + blockIdx.x] = s;   // digit-major: one contiguous row per digit
}

// Per digit (one CTA each): exclusive scan of the row of per-block counts, in place, and the row
// total.  Done once per pass here instead of by every scatter CTA.
__global__ void __launch_bounds__(256) k_radix_scan_rows(uint32_t *__restrict__ table, int nblocks,
                                                         uint32_t *__restrict__ totals) {
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

__device__ __forceinline__ uint32_t block_exclusive_scan_256(uint32_t v, uint32_t *s_warp_tot, int tid) {
  const int lane = tid & 31, warp = tid >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t t = __shfl_up_sync(kFull, inc, s);
    if (lane >= s) inc += t;
  }
  if (lane == 31) s_warp_tot[warp] = inc;
  __syncthreads();
  uint32_t off = 0;
#pragma unroll
  for (int w = 0; w < kSortWarps; ++w) off += (w < warp) ? s_warp_tot[w] : 0u;
  __syncthreads();
  return off + inc - v;
}

// One pass: stable scatter of this block's range by the BITS-wide digit at `shift`.  Slots past the
// end of the input carry the largest digit and sit at the end of the last tile, so they rank after
// every real key and are never written.
// EP selects the epilogue: 0 none, 1 block sums of tiles touched (last pass of the depth sort), 2 tile ranges (last
// pass of the tile sort: inside a block's run of one digit the keys are non-decreasing, because the earlier passes
// ordered the lower bits, so a change of key between neighbours of a run is a tile boundary; the two ends of a run
// may continue in another block and enter with an atomic min / max).
template <int BITS, int EP>
__global__ void __launch_bounds__(kSortThreads, 3) k_radix_scatter(
    const uint32_t *__restrict__ keys_in, const uint32_t *__restrict__ vals_in, uint32_t *__restrict__ keys_out,
    uint32_t *__restrict__ vals_out, int64_t count, const unsigned long long *__restrict__ count_dev, int shift,
    int tiles_per_block, int extra,
    const uint32_t *__restrict__ table, const uint32_t *__restrict__ totals, int nblocks, SortEpilogue ep) {
  __shared__ uint32_t s_keys[kSortTile];
  __shared__ uint32_t s_vals[kSortTile];
  __shared__ uint32_t s_warp_cnt[kSortWarps][256];
  __shared__ uint32_t s_digit_start[256];
  __shared__ uint32_t s_base[256];
  __shared__ uint32_t s_warp_tot[kSortWarps];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t lt_mask = (1u << lane) - 1u;
  if (count_dev) count = min(count, (int64_t)__ldg(count_dev));
  constexpr uint32_t kDigitMask = (1u << BITS) - 1u;

  // global base of every digit for this block: all smaller digits everywhere (scan of the row
  // totals) + the same digit in the blocks before this one (the row prefix from k_radix_scan_rows)
  {
    const uint32_t start = block_exclusive_scan_256(__ldg(totals + tid), s_warp_tot, tid);
    s_base[tid] = start + __ldg(table + (size_t)tid * nblocks + blockIdx.x);
  }

  int64_t first_tile;
  int my_tiles;
  block_tiles(tiles_per_block, extra, first_tile, my_tiles);
  const int64_t begin = first_tile * kSortTile;
  for (int t = 0; t < my_tiles; ++t) {
    const int64_t tile_begin = begin + (int64_t)t * kSortTile;
    if (tile_begin >= count) break;
    const int valid_count = (int)min((int64_t)kSortTile, count - tile_begin);
    for (int k = tid; k < kSortWarps * 256; k += kSortThreads) (&s_warp_cnt[0][0])[k] = 0;
    __syncthreads();
    uint32_t key[kItems], val[kItems];
    unsigned short rank[kItems];
    // all loads first (independent, in flight together), then the serial ranking chain
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int local = warp * (32 * kItems) + it * 32 + lane;
      const bool ok = local < valid_count;
      const int64_t idx = tile_begin + local;
      key[it] = ok ? __ldg(keys_in + idx) : 0xffffffffu;
      val[it] = ok ? (vals_in ? __ldg(vals_in + idx) : (uint32_t)idx) : 0u;
    }
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int local = warp * (32 * kItems) + it * 32 + lane;
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
      if (lane == leader) prior = atomicAdd(&s_warp_cnt[warp][d], (uint32_t)__popc(peers));
      prior = __shfl_sync(kFull, prior, leader);
      rank[it] = (unsigned short)(prior + __popc(peers & lt_mask));
    }
    __syncthreads();
    // per digit: exclusive scan over warps, then over digits
    uint32_t cnt = 0;
#pragma unroll
    for (int w = 0; w < kSortWarps; ++w) {
      const uint32_t c = s_warp_cnt[w][tid];
      s_warp_cnt[w][tid] = cnt;
      cnt += c;
    }
    const uint32_t dstart = block_exclusive_scan_256(cnt, s_warp_tot, tid);
    s_digit_start[tid] = dstart;
    __syncthreads();
#pragma unroll
    for (int it = 0; it < kItems; ++it) {
      const int local = warp * (32 * kItems) + it * 32 + lane;
      const uint32_t d = (local < valid_count) ? ((key[it] >> shift) & kDigitMask) : kDigitMask;
      const uint32_t pos = s_digit_start[d] + s_warp_cnt[warp][d] + rank[it];
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
        // tiles touched by this Gaussian, added to the sum of its block of kScanBlock sorted positions; a warp whose
        // lanes all fall into one block (the usual case: a run is contiguous) adds once
        uint32_t tt = ok ? __ldg(ep.tiles_touched + v) : 0u;
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
        if ((uint32_t)j == run_first) atomicMin(ep.ranges + 2 * k, gpos);
        else if (s_keys[j - 1] != k) ep.ranges[2 * k] = gpos;
        if ((uint32_t)j + 1 == run_end) atomicMax(ep.ranges + 2 * k + 1, gpos + 1);
        else if (s_keys[j + 1] != k) ep.ranges[2 * k + 1] = gpos + 1;
      }
    }
    __syncthreads();
    s_base[tid] += cnt;
    __syncthreads();
  }
}

// ---- tiles touched in depth order -----------------------------------------------------------

// Emit the instances of each Gaussian, in depth order: the tiles its alpha >= 1/255 ellipse meets
// (TileSpans, the same function the preprocess counted with), tile rows top to bottom, tiles left
// to right.  Small footprints are written by their own thread; large ones by the whole warp.
constexpr uint32_t kKeygenStage = 512;   // instances a warp stages in shared memory (4 KB per warp)

__global__ void __launch_bounds__(kScanBlock) k_keygen(const uint32_t *__restrict__ order, const uint16_t *__restrict__ rect,
                                                       const float *__restrict__ mean2d,
                                                       const float *__restrict__ conic_opacity,
                                                       const uint32_t *__restrict__ tiles_touched,
                                                       const uint32_t *__restrict__ block_sums, int64_t n, int gx,
                                                       int W, int H, uint32_t capacity,
                                                       uint32_t *__restrict__ inst_tiles,
                                                       uint32_t *__restrict__ inst_vals) {
  __shared__ uint32_t s_w[kScanBlock / 32], s_before[kScanBlock / 32];
  __shared__ uint32_t s_stage[kScanBlock / 32][2 * kKeygenStage];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t i = (int64_t)blockIdx.x * kScanBlock + tid;
  uint32_t g = 0, tiles = 0;
  ushort4 r = make_ushort4(0, 0, 0, 0);
  float4 sp0 = make_float4(0.f, 0.f, 1.f, 0.f);   // u, v, la, lb
  float2 sp1 = make_float2(1.f, 0.f);             // lc, tau
  if (i < n) {
    g = __ldg(order + i);
    // the four gathers go out together (also for Gaussians without tiles, whose rows are then ignored)
    tiles = __ldg(tiles_touched + g);
    const ushort4 rr = __ldg(reinterpret_cast<const ushort4 *>(rect) + g);
    const float2 m = __ldg(reinterpret_cast<const float2 *>(mean2d) + g);
    const float4 q = __ldg(reinterpret_cast<const float4 *>(conic_opacity) + g);
    if (tiles) {
      r = rr;
      sp0 = make_float4(m.x, m.y, q.x, q.y);
      sp1 = make_float2(q.z, footprint_tau(q.w));
    }
  }
  uint32_t inc = tiles;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t t = __shfl_up_sync(kFull, inc, s);
    if (lane >= s) inc += t;
  }
  if (lane == 31) s_w[warp] = inc;
  // instances of all CTAs before this one: the sums per kScanBlock Gaussians come from the last pass of the depth
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
  off += inc - tiles;
  constexpr uint32_t kSmall = 32;
  // A warp whose footprints add up to at most kKeygenStage instances writes them to shared memory first and
  // copies the block out with coalesced stores; lanes writing their own short runs directly would touch a
  // different sector with every store.  Staged or not, the emission below is the same: only the destination
  // and the origin of the positions differ.
  const uint32_t warp_total = __shfl_sync(kFull, inc, 31);
  const uint32_t warp_base = __shfl_sync(kFull, off, 0);
  const bool staged = warp_total <= kKeygenStage;
  uint32_t *dst_tiles = staged ? s_stage[warp] : inst_tiles;
  uint32_t *dst_vals = staged ? s_stage[warp] + kKeygenStage : inst_vals;
  const uint32_t limit = staged ? kKeygenStage : capacity;   // never past the buffers, even if the count was taken on the device
  if (staged) off -= warp_base;
  if (tiles > 0 && tiles <= kSmall) {
    TileSpans sp;
    sp.setup(sp0.x, sp0.y, sp0.z, sp0.w, sp1.x, sp1.y, W, H);
    uint32_t p = off;
    for (int ty = r.y; ty < (int)r.w; ++ty) {
      int xa, xb;
      if (!sp.row(ty, r.x, r.z, xa, xb)) continue;
      for (int tx = xa; tx < xb; ++tx) {
        if (p < limit) {
          dst_tiles[p] = (uint32_t)(ty * gx + tx);
          dst_vals[p] = g;
        }
        ++p;
      }
    }
  }
  // a large footprint is shared by the warp: one tile row per lane, then the tiles of each row
  uint32_t big = __ballot_sync(kFull, tiles > kSmall);
  while (big) {
    const int src = __ffs(big) - 1;
    big &= big - 1;
    TileSpans sp;
    sp.setup(__shfl_sync(kFull, sp0.x, src), __shfl_sync(kFull, sp0.y, src), __shfl_sync(kFull, sp0.z, src),
             __shfl_sync(kFull, sp0.w, src), __shfl_sync(kFull, sp1.x, src), __shfl_sync(kFull, sp1.y, src), W, H);
    uint32_t p = __shfl_sync(kFull, off, src);
    const uint32_t s_g = __shfl_sync(kFull, g, src);
    const int x0 = (int)__shfl_sync(kFull, (uint32_t)r.x, src), x1 = (int)__shfl_sync(kFull, (uint32_t)r.z, src);
    const int y0 = (int)__shfl_sync(kFull, (uint32_t)r.y, src), y1 = (int)__shfl_sync(kFull, (uint32_t)r.w, src);
    for (int tyb = y0; tyb < y1; tyb += 32) {
      int xa = 0, xb = 0;
      if (tyb + lane < y1 && !sp.row(tyb + lane, x0, x1, xa, xb)) xa = xb = 0;
      uint32_t incl = (uint32_t)(xb - xa);
#pragma unroll
      for (int s = 1; s < 32; s <<= 1) {
        const uint32_t t = __shfl_up_sync(kFull, incl, s);
        if (lane >= s) incl += t;
      }
      const uint32_t excl = incl - (uint32_t)(xb - xa);
      const int rows = min(32, y1 - tyb);
      for (int rr = 0; rr < rows; ++rr) {
        const int a = __shfl_sync(kFull, xa, rr), b = __shfl_sync(kFull, xb, rr);
        const uint32_t o = p + __shfl_sync(kFull, excl, rr);
        for (int tx = a + lane; tx < b; tx += 32) {
          const uint32_t q = o + (uint32_t)(tx - a);
          if (q < limit) {
            dst_tiles[q] = (uint32_t)((tyb + rr) * gx + tx);
            dst_vals[q] = s_g;
          }
        }
      }
      p += __shfl_sync(kFull, incl, 31);
    }
  }
  if (staged) {
    __syncwarp();
    const uint32_t *st = s_stage[warp], *sv = st + kKeygenStage;
    for (uint32_t q = lane; q < warp_total; q += 32) {
      if (warp_base + q < capacity) {
        inst_tiles[warp_base + q] = st[q];
        inst_vals[warp_base + q] = sv[q];
      }
    }
  }
}

// Launch order of the blend CTAs: tiles by decreasing list length (log2 buckets), so that the long
// tiles start first and the short ones fill the tail.  The order inside a bucket is whatever the
// atomics give; it affects scheduling only, never a result.
// A tile without instances comes in as (0xffffffff, 0), the neutral values of the range epilogue, and leaves as (0, 0).
__global__ void __launch_bounds__(1024) k_tile_order(uint32_t *__restrict__ ranges, int num_tiles,
                                                     uint32_t *__restrict__ order) {
  __shared__ uint32_t s_cnt[33], s_off[33];
  const int tid = threadIdx.x;
  if (tid < 33) s_cnt[tid] = 0;
  __syncthreads();
  for (int t = tid; t < num_tiles; t += 1024) {
    if (ranges[2 * t + 1] == 0u) ranges[2 * t] = 0u;
    const uint32_t len = ranges[2 * t + 1] - ranges[2 * t];
    atomicAdd(&s_cnt[len ? 32 - __clz(len) : 0], 1u);
  }
  __syncthreads();
  if (tid == 0) {
    uint32_t off = 0;
    for (int b = 32; b >= 0; --b) { s_off[b] = off; off += s_cnt[b]; }
  }
  __syncthreads();
  for (int t = tid; t < num_tiles; t += 1024) {
    const uint32_t len = ranges[2 * t + 1] - ranges[2 * t];
    order[atomicAdd(&s_off[len ? 32 - __clz(len) : 0], 1u)] = (uint32_t)t;
  }
}

}  // namespace

size_t sort_scratch_bytes(int64_t count) { return ((size_t)plan_for(count).blocks + 1) * 256 * sizeof(uint32_t); }

int launch_radix_sort(const uint32_t *keys_in, const uint32_t *vals_in, uint32_t *keys_out, uint32_t *vals_out,
                       uint32_t *tmp_keys, uint32_t *tmp_vals, int64_t count, const unsigned long long *count_dev,
                       int num_bits, void *scratch, const SortEpilogue *epilogue, cudaStream_t st) {
  if (count <= 0) return 0;
  const SortPlan plan = plan_for(count);
  int passes = (num_bits + 7) / 8;
  if (passes < 1) passes = 1;
  const int bits = (num_bits + passes - 1) / passes;     // digits of equal width: 13 bits sort as 7 + 6
  uint32_t *table = static_cast<uint32_t *>(scratch);
  uint32_t *totals = table + (size_t)plan.blocks * 256;
  const uint32_t *src_k = keys_in, *src_v = vals_in;
  const SortEpilogue none = {nullptr, nullptr, 0, nullptr, 0, nullptr};
  for (int p = 0; p < passes; ++p) {
    const bool to_out = ((passes - 1 - p) % 2) == 0;
    uint32_t *dst_k = to_out ? keys_out : tmp_keys, *dst_v = to_out ? vals_out : tmp_vals;
    const SortEpilogue ep = (p == passes - 1 && epilogue) ? *epilogue : none;
    const int mode = ep.block_sums ? 1 : ep.ranges ? 2 : 0;
    k_radix_hist<<<plan.blocks, kSortThreads, 0, st>>>(src_k, count, count_dev, bits * p, (1u << bits) - 1u,
                                                        plan.tiles_per_block, plan.extra, table, ep);
    k_radix_scan_rows<<<256, 256, 0, st>>>(table, plan.blocks, totals);
#define GS_SCATTER_ARGS                                                                                              \
  <<<plan.blocks, kSortThreads, 0, st>>>(src_k, src_v, dst_k, dst_v, count, count_dev, bits * p, plan.tiles_per_block, \
                                         plan.extra, table, totals, plan.blocks, ep)
#define GS_SCATTER(B)                                              \
  case B:                                                          \
    if (mode == 2) k_radix_scatter<B, 2> GS_SCATTER_ARGS;          \
    else k_radix_scatter<B, 0> GS_SCATTER_ARGS;                    \
    break;
    switch (bits) {
      GS_SCATTER(1) GS_SCATTER(2) GS_SCATTER(3) GS_SCATTER(4) GS_SCATTER(5) GS_SCATTER(6) GS_SCATTER(7)
      default:
        if (mode == 1) k_radix_scatter<8, 1> GS_SCATTER_ARGS;
        else if (mode == 2) k_radix_scatter<8, 2> GS_SCATTER_ARGS;
        else k_radix_scatter<8, 0> GS_SCATTER_ARGS;
    }
#undef GS_SCATTER
#undef GS_SCATTER_ARGS
    src_k = dst_k;
    src_v = dst_v;
  }
  return 3 * passes;
}

size_t scan_scratch_bytes(int64_t n) { return (size_t)((n + kScanBlock - 1) / kScanBlock + 1) * sizeof(uint32_t); }
int num_scan_blocks(int64_t n) { return (int)((n + kScanBlock - 1) / kScanBlock); }

int launch_keygen(const uint32_t *depth_order, const uint16_t *rect, const float *mean2d, const float *conic_opacity,
                  const uint32_t *tiles_touched, const uint32_t *block_sums, uint32_t *inst_tiles, uint32_t *inst_vals,
                  int64_t n, int gx, int W, int H, int64_t capacity, cudaStream_t st) {
  if (n <= 0) return 0;
  const int blocks = num_scan_blocks(n);
  const uint32_t cap = capacity > 0xffffffffll ? 0xffffffffu : (uint32_t)capacity;
  k_keygen<<<blocks, kScanBlock, 0, st>>>(depth_order, rect, mean2d, conic_opacity, tiles_touched, block_sums, n, gx, W, H,
                                          cap, inst_tiles, inst_vals);
  return 1;
}

// Settles the ranges of the empty tiles and orders the tiles for the blend launches.  With `clear` (no instance was
// sorted, so no range epilogue ran) every range is zeroed first.
int launch_tile_order(uint32_t *ranges, uint32_t *order, int num_tiles, bool clear, cudaStream_t st) {
  if (clear) cudaMemsetAsync(ranges, 0, (size_t)num_tiles * 2 * sizeof(uint32_t), st);
  k_tile_order<<<1, 1024, 0, st>>>(ranges, num_tiles, order);
  return 1;
}

}  // namespace gs

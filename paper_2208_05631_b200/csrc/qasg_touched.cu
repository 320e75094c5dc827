// Passes A and B for gradients held in sparse form: a worker's row stores only the entries its touched
// bits mark, every other entry is +0.0 and its memory is never read.
//
// One WARP takes a whole tile (4 rows x 1024 columns): lane l owns the 32 columns 32l .. 32l+31, i.e. one
// word of touched bits per row, so a tile without entries costs four coalesced word loads and a vote, and a
// stored entry costs one scalar load.  The sums are those of the dense kernels bit for bit, because the
// tree is the same and adding +0.0 changes nothing: column sums down the rows, a pairwise tree over a
// lane's 32 columns (levels 0-4), the lane butterfly (levels 5-9), a pairwise tree over the tiles of a
// chunk (one warp per batch of up to 64 tiles, a pairwise stack over the batches), chunk partials combined
// by the last CTA.  A lane takes one of three paths by the number of its touched columns: one or two (the
// usual case: all loads issued together, a + b is the tree), up to twelve (column after column, the next
// column's loads ahead), more (the head of a row whose column frequencies are Zipf-like is full: 128-bit
// loads of all four rows in flight together, values and column sums in local memory).  Rows that are full
// throughout are better served by the dense entry points.  A tile with more than kCrowdedTile entries is walked
// in the dense layout instead (crowded_tile below).  (Capping the registers to keep five CTAs per SM made the
// crowded path spill and every pattern slower.)
#include "qasg_device.cuh"

namespace qasg {

namespace {

constexpr int kWarps = kThreads / 32;
constexpr int kTouchedBatch = 64;  // tiles between two meetings of the CTA (a warp takes every eighth of them)

struct TouchedStorage {
  double tile_sums[kTouchedBatch];
  double stack[32];
};

// The four words of touched bits of lane `lane` for tile k (row r: columns 32*lane .. 32*lane+31).
// Bits at or past d are dropped, so nothing at or past d is ever loaded.
__device__ __forceinline__ void load_lane_words(const uint32_t* __restrict__ trow, uint64_t d, uint32_t k, int lane,
                                                bool ragged, uint32_t (&w)[kTileRows]) {
#pragma unroll
  for (int r = 0; r < kTileRows; ++r) {
    const uint64_t idx = static_cast<uint64_t>(k) * (kTile / 32) + r * (kTileCols / 32) + lane;
    if (!ragged) {
      w[r] = __ldg(trow + idx);
    } else if (idx * 32 < d) {
      w[r] = __ldg(trow + idx);
      if (d - idx * 32 < 32) w[r] &= (1u << (d - idx * 32)) - 1u;
    } else {
      w[r] = 0u;
    }
  }
}

// Pairwise (adjacent-pair) tree over a lane's 32 column sums.
__device__ __forceinline__ double lane_tree(double (&col)[32]) {
#pragma unroll
  for (int s = 1; s < 32; s <<= 1)
#pragma unroll
    for (int i = 0; i < 32; i += 2 * s) col[i] += col[i + s];
  return col[0];
}

// Walks the stored entries of the lane's 32 columns of one tile, column by column, rows in order:
// entry(r, c, value) returns the magnitude that enters the column's sum (+0.0 for "not kept").
// Returns the lane's sum in tree order.  One or two non-zero columns need no tree (a + b is the tree).
template <class Entry>
__device__ __forceinline__ double lane_columns(const float* __restrict__ row, uint64_t tile_base, int lane,
                                               const uint32_t (&w)[kTileRows], Entry&& entry) {
  uint32_t cols = (w[0] | w[1]) | (w[2] | w[3]);
  if (!cols) return 0.0;
  const int n = __popc(cols);
  const float* base = row + tile_base + 32 * lane;
  if (n <= 2) {  // the usual case: all (up to eight) loads are issued before any is used
    const int c0 = __ffs(cols) - 1;
    const uint32_t rest = cols & (cols - 1);
    const int c1 = rest ? __ffs(rest) - 1 : c0;
    float v0[kTileRows], v1[kTileRows];
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      v0[r] = ((w[r] >> c0) & 1u) ? __ldg(base + r * kTileCols + c0) : 0.f;
      v1[r] = (rest && ((w[r] >> c1) & 1u)) ? __ldg(base + r * kTileCols + c1) : 0.f;
    }
    double acc0 = 0.0, acc1 = 0.0;
#pragma unroll
    for (int r = 0; r < kTileRows; ++r)
      if ((w[r] >> c0) & 1u) acc0 += static_cast<double>(entry(r, c0, v0[r]));
    if (rest) {
#pragma unroll
      for (int r = 0; r < kTileRows; ++r)
        if ((w[r] >> c1) & 1u) acc1 += static_cast<double>(entry(r, c1, v1[r]));
    }
    return acc0 + acc1;
  }
  double col[32];
  if (n <= 12) {  // a few columns: one after the other, the next column's values requested ahead
#pragma unroll
    for (int c = 0; c < 32; ++c) col[c] = 0.0;
    auto fetch = [&](int c, float (&v)[kTileRows]) {
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) v[r] = ((w[r] >> c) & 1u) ? __ldg(base + r * kTileCols + c) : 0.f;
    };
    float v[kTileRows], vn[kTileRows] = {0.f, 0.f, 0.f, 0.f};
    int c = __ffs(cols) - 1;
    uint32_t rest = cols & (cols - 1);
    fetch(c, v);
    while (true) {
      const int cn = rest ? __ffs(rest) - 1 : -1;
      if (cn >= 0) {
        rest &= rest - 1;
        fetch(cn, vn);
      }
      double acc = 0.0;
#pragma unroll
      for (int r = 0; r < kTileRows; ++r)
        if ((w[r] >> c) & 1u) acc += static_cast<double>(entry(r, c, v[r]));
      col[c] = acc;
      if (cn < 0) break;
      c = cn;
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) v[r] = vn[r];
    }
    return lane_tree(col);
  }
  // A crowded lane: the float4 of its 4 x 32 coordinates that hold an entry are all requested together and
  // parked in local memory; the columns are then taken one by one (dynamic indices: the values and the 32
  // column sums live in local memory, which keeps the registers of the common path low).
  float vals[kTileRows][32];
#pragma unroll
  for (int r = 0; r < kTileRows; ++r) {
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const float4 v = ((w[r] >> (4 * q)) & 15u) ? load_f4(base + r * kTileCols + 4 * q) : make_float4(0.f, 0.f, 0.f, 0.f);
      *reinterpret_cast<float4*>(&vals[r][4 * q]) = v;
    }
  }
#pragma unroll 1
  for (int c = 0; c < 32; ++c) {
    double acc = 0.0;
#pragma unroll
    for (int r = 0; r < kTileRows; ++r)
      if ((w[r] >> c) & 1u) acc += static_cast<double>(entry(r, c, vals[r][c]));
    col[c] = acc;
  }
  return lane_tree(col);
}

// A crowded tile (more than kCrowdedTile entries), still by one warp, in the dense kernels' layout: eight
// slices of 128 columns; in slice q lane l takes the float4 at columns 128q + 4l .. + 3 of each row whose
// nibble of bits is non-zero (untouched lanes forced to +0.0).  slice(values, nibbles, q) returns the
// thread's share (cx + cy) + (cz + cw) of the slice; the lane butterfly makes it the sum of the slice's 128
// columns (levels 0-6 of the tree) and the eight slices are combined pairwise (levels 7-9).
constexpr uint32_t kCrowdedTile = 128;

__device__ __forceinline__ uint32_t tile_entries(const uint32_t (&w)[kTileRows]) {
  return __reduce_add_sync(0xffffffffu, (__popc(w[0]) + __popc(w[1])) + (__popc(w[2]) + __popc(w[3])));
}

template <class Slice>
__device__ __forceinline__ double crowded_tile(const float* __restrict__ row, uint64_t tile_base, int lane,
                                               const uint32_t (&w)[kTileRows], Slice&& slice) {
  double s0 = 0.0, s1 = 0.0, s2 = 0.0, total = 0.0;  // pairwise stack over the slices
#pragma unroll 1
  for (int q = 0; q < 8; ++q) {
    uint32_t nibs = 0u;
    float4 v[kTileRows];
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      const uint32_t word = __shfl_sync(0xffffffffu, w[r], 4 * q + (lane >> 3));
      const uint32_t nib = (word >> (4 * (lane & 7))) & 15u;
      nibs |= nib << (4 * r);
      float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
      if (nib) {  // some coordinate below d is marked: the float4 lies inside the row
        t = load_f4(row + tile_base + r * kTileCols + 128 * q + 4 * lane);
        if (!(nib & 1u)) t.x = 0.f;
        if (!(nib & 2u)) t.y = 0.f;
        if (!(nib & 4u)) t.z = 0.f;
        if (!(nib & 8u)) t.w = 0.f;
      }
      v[r] = t;
    }
    double x = warp_pair_tree(slice(v, nibs, q));
    if (q & 1) {
      x = s0 + x;
      if (q & 2) {
        x = s1 + x;
        if (q & 4) total = s2 + x;
        else s2 = x;
      } else {
        s1 = x;
      }
    } else {
      s0 = x;
    }
  }
  return total;
}

// The tiles of the CTA's items, one warp per tile, in batches of kTouchedBatch tiles:
//   begin(m, c)                    all threads, before an item
//   tile(m, k, words) -> double    one warp, a tile with entries: its sum (valid in every lane)
//   empty(m, k)                    one warp, a tile without entries
//   end(m, c, chunk_sum)           all threads, after an item; chunk_sum is valid in thread 0
template <class Begin, class Tile, class Empty, class End>
__device__ __forceinline__ void stream_touched_tiles(const uint32_t* __restrict__ touched, const Geometry& geo,
                                                     TouchedStorage* st, Begin&& begin, Tile&& tile, Empty&& empty,
                                                     End&& end) {
  const int j = threadIdx.x, warp = j >> 5, lane = j & 31;
  const uint32_t n_items = geo.M * geo.chunks;
  const uint64_t words = (geo.d + 31) >> 5;
  const uint32_t ragged_tile = (geo.d % kTile) ? geo.tiles - 1 : 0xffffffffu;
  for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const ItemPos p = item_pos(geo, item);
    const uint32_t* trow = touched + static_cast<uint64_t>(p.m) * words;
    begin(p.m, p.c);
    uint32_t pushed = 0;
    for (uint32_t base = p.k0; base < p.k1; base += kTouchedBatch) {
      const uint32_t batch = min(static_cast<uint32_t>(kTouchedBatch), p.k1 - base);
      uint32_t w[kTileRows] = {0u, 0u, 0u, 0u}, wn[kTileRows] = {0u, 0u, 0u, 0u};
      if (static_cast<uint32_t>(warp) < batch) load_lane_words(trow, geo.d, base + warp, lane, base + warp == ragged_tile, w);
      for (uint32_t t = warp; t < batch; t += kWarps) {
        const uint32_t k = base + t;
        if (t + kWarps < batch) load_lane_words(trow, geo.d, k + kWarps, lane, k + kWarps == ragged_tile, wn);
        double s = 0.0;
        if (__any_sync(0xffffffffu, ((w[0] | w[1]) | (w[2] | w[3])) != 0u)) s = tile(p.m, k, w);
        else empty(p.m, k);
        if (lane == 0) st->tile_sums[t] = s;
#pragma unroll
        for (int r = 0; r < kTileRows; ++r) w[r] = wn[r];
      }
      __syncthreads();
      // The batch is an aligned block of up to 64 tiles, i.e. a complete subtree of the pairwise tree over
      // tiles (missing tiles count +0.0): one warp sums it - adjacent pairs inside a lane, then the lane
      // butterfly - and one value per batch goes onto the stack.  (A serial push of every tile by one
      // thread, with the CTA waiting, cost more than the tiles themselves.)
      if (warp == 0) {
        const double a = 2u * lane < batch ? st->tile_sums[2 * lane] : 0.0;
        const double b = 2u * lane + 1 < batch ? st->tile_sums[2 * lane + 1] : 0.0;
        const double batch_sum = warp_pair_tree(a + b);
        if (lane == 0) tile_push(st->stack, pushed, batch_sum);
      }
      ++pushed;
      __syncthreads();
    }
    double total = 0.0;
    // the stack holds batches: log2(batches per chunk) levels
    if (j == 0) total = tile_fold(st->stack, pushed, geo.log2_group > 6 ? geo.log2_group - 6 : 0);
    end(p.m, p.c, total);
  }
}

// ------------------------------------------------------------------ pass A
__global__ void __launch_bounds__(kThreads)
touched_abs_sum_kernel(const float* __restrict__ g, Geometry geo, float coef, Workspace ws,
                       float* __restrict__ thresholds_out, const uint32_t* __restrict__ touched) {
  __shared__ TouchedStorage st;
  __shared__ bool sm_last;
  const int j = threadIdx.x, lane = j & 31;
  stream_touched_tiles(
      touched, geo, &st, [](uint32_t, uint32_t) {},
      [&](uint32_t m, uint32_t k, const uint32_t (&w)[kTileRows]) -> double {
        const float* row = g + static_cast<uint64_t>(m) * geo.ld;
        if (tile_entries(w) > kCrowdedTile)
          return crowded_tile(row, static_cast<uint64_t>(k) * kTile, lane, w,
                              [](const float4 (&v)[kTileRows], uint32_t, int) -> double {
                                double cx = fabsf(v[0].x), cy = fabsf(v[0].y), cz = fabsf(v[0].z), cw = fabsf(v[0].w);
#pragma unroll
                                for (int r = 1; r < kTileRows; ++r) {
                                  cx += static_cast<double>(fabsf(v[r].x));
                                  cy += static_cast<double>(fabsf(v[r].y));
                                  cz += static_cast<double>(fabsf(v[r].z));
                                  cw += static_cast<double>(fabsf(v[r].w));
                                }
                                return (cx + cy) + (cz + cw);
                              });
        const double s = lane_columns(row, static_cast<uint64_t>(k) * kTile, lane, w, [](int, int, float v) { return fabsf(v); });
        return warp_pair_tree(s);
      },
      [](uint32_t, uint32_t) {},
      [&](uint32_t m, uint32_t c, double total) {
        if (j == 0) ws.part_sum[static_cast<uint64_t>(m) * kMaxChunks + c] = total;
      });
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  const int warp = j >> 5;
  for (uint32_t m = warp; m < geo.M; m += kWarps) {
    const double total = warp_chunk_tree(ws.part_sum + static_cast<uint64_t>(m) * kMaxChunks, geo.chunks, lane);
    if (lane == 0) {
      const float delta = static_cast<float>((static_cast<double>(coef) * total) / static_cast<double>(geo.d));
      ws.thresholds[m] = delta;
      if (thresholds_out) thresholds_out[m] = delta;
      if (!isfinite(total)) atomicOr(ws.status, kFlagNonFinite);
    }
  }
  if (j == 0) *ws.ticket = 0u;
}

// ------------------------------------------------------------------ pass A': max |g|
__global__ void __launch_bounds__(kThreads)
touched_abs_max_kernel(const float* __restrict__ g, Geometry geo, Workspace ws, const uint32_t* __restrict__ touched) {
  __shared__ TouchedStorage st;
  __shared__ uint32_t sm_warp[kWarps];
  __shared__ bool sm_last;
  const int j = threadIdx.x, lane = j & 31, warp = j >> 5;
  uint32_t best = 0u;  // this thread's maximum over the current item
  stream_touched_tiles(
      touched, geo, &st, [&](uint32_t, uint32_t) { best = 0u; },
      [&](uint32_t m, uint32_t k, const uint32_t (&w)[kTileRows]) -> double {
        const float* row = g + static_cast<uint64_t>(m) * geo.ld;
        if (tile_entries(w) > kCrowdedTile) {
          crowded_tile(row, static_cast<uint64_t>(k) * kTile, lane, w,
                       [&](const float4 (&v)[kTileRows], uint32_t, int) -> double {
#pragma unroll
                         for (int r = 0; r < kTileRows; ++r) {  // untouched lanes are +0.0 and change no maximum
                           best = max(best, __float_as_uint(fabsf(v[r].x)));
                           best = max(best, __float_as_uint(fabsf(v[r].y)));
                           best = max(best, __float_as_uint(fabsf(v[r].z)));
                           best = max(best, __float_as_uint(fabsf(v[r].w)));
                         }
                         return 0.0;
                       });
          return 0.0;
        }
        lane_columns(row, static_cast<uint64_t>(k) * kTile, lane, w, [&](int, int, float v) {
          best = max(best, __float_as_uint(fabsf(v)));
          return 0.f;
        });
        return 0.0;
      },
      [](uint32_t, uint32_t) {},
      [&](uint32_t m, uint32_t c, double) {
        const uint32_t wbest = __reduce_max_sync(0xffffffffu, best);
        if (lane == 0) sm_warp[warp] = wbest;
        __syncthreads();
        if (j == 0) {
          uint32_t bmax = sm_warp[0];
#pragma unroll
          for (int q = 1; q < kWarps; ++q) bmax = max(bmax, sm_warp[q]);
          ws.part_max[static_cast<uint64_t>(m) * kMaxChunks + c] = bmax;
        }
        __syncthreads();
      });
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  for (uint32_t m = warp; m < geo.M; m += kWarps) {
    uint32_t bmax = 0u;
    for (uint32_t idx = lane; idx < geo.chunks; idx += 32)
      bmax = max(bmax, __ldcg(ws.part_max + static_cast<uint64_t>(m) * kMaxChunks + idx));
    bmax = __reduce_max_sync(0xffffffffu, bmax);
    if (lane == 0) {
      ws.scales[m] = __uint_as_float(bmax);
      ws.thresholds[m] = 0.f;
      if (bmax >= 0x7f800000u) atomicOr(ws.status, kFlagNonFinite);
    }
  }
  if (j == 0) *ws.ticket = 0u;
}

// ------------------------------------------------------------------ pass B (both quantizers)
// A lane's code bits of one tile: per row 32 coordinates = 64 bits = two words of the code row, at word
// offset k*256 + r*64 + 2*lane.  Everything that is not stored codes 0.
struct LaneCodes {
  uint32_t lo[kTileRows], hi[kTileRows];
  __device__ __forceinline__ void clear() {
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) lo[r] = hi[r] = 0u;
  }
  __device__ __forceinline__ void set(int r, int c, uint32_t code) {
    // r is a compile-time index at every call site (unrolled row loop)
    if (c < 16) lo[r] |= code << (2 * c);
    else hi[r] |= code << (2 * (c - 16));
  }
  // wide: the code row starts on an 8-byte boundary (an even number of words per row), so a lane's two
  // words of a row leave as one 64-bit store.
  __device__ __forceinline__ void store(uint32_t* __restrict__ code_row, uint64_t row_words, uint32_t k, int lane,
                                        bool wide) const {
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      const uint64_t off = static_cast<uint64_t>(k) * (kTile / 16) + r * (kTileCols / 16) + 2 * lane;
      if (wide) {
        if (off < row_words) __stcs(reinterpret_cast<uint2*>(code_row + off), make_uint2(lo[r], hi[r]));
      } else {
        if (off < row_words) __stcs(code_row + off, lo[r]);
        if (off + 1 < row_words) __stcs(code_row + off + 1, hi[r]);
      }
    }
  }
};

template <bool kStochastic>
__global__ void __launch_bounds__(kThreads)
touched_codes_kernel(const float* __restrict__ g, Geometry geo, uint64_t seed, uint64_t t, uint32_t stream_base,
                     Workspace ws, uint32_t* __restrict__ codes, float* __restrict__ scales_out,
                     unsigned long long* __restrict__ counts_out, const uint32_t* __restrict__ touched) {
  __shared__ TouchedStorage st;
  __shared__ uint32_t sm_cnt[kWarps];
  __shared__ bool sm_last;
  const int j = threadIdx.x, lane = j & 31;
  const uint64_t row_words = (geo.d + 15) >> 4;
  const bool wide = (row_words & 1u) == 0 && (reinterpret_cast<uintptr_t>(codes) & 7u) == 0;
  const uint32_t key0 = static_cast<uint32_t>(seed), key1 = static_cast<uint32_t>(seed >> 32);
  const uint32_t t_lo = static_cast<uint32_t>(t), t_hi = static_cast<uint32_t>(t >> 32);
  float delta = 0.f, ndelta = 0.f, scale = 0.f;
  uint32_t cnt = 0;
  stream_touched_tiles(
      touched, geo, &st,
      [&](uint32_t m, uint32_t) {
        delta = ws.thresholds[m];
        ndelta = -delta;
        scale = ws.scales[m];  // stochastic quantizer: the maximum found by pass A'
        cnt = 0;
      },
      [&](uint32_t m, uint32_t k, const uint32_t (&w)[kTileRows]) -> double {
        const uint64_t tile_base = static_cast<uint64_t>(k) * kTile;
        if (tile_entries(w) > kCrowdedTile) {
          uint8_t* codes8 = reinterpret_cast<uint8_t*>(codes + static_cast<uint64_t>(m) * row_words);
          const double s = crowded_tile(
              g + static_cast<uint64_t>(m) * geo.ld, tile_base, lane, w,
              [&](const float4 (&v)[kTileRows], uint32_t nibs, int q) -> double {
                double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
#pragma unroll
                for (int r = 0; r < kTileRows; ++r) {
                  const float4 t = v[r];
                  uint32_t byte = 0u;
                  if ((nibs >> (4 * r)) & 15u) {
                    if (!kStochastic) {
                      const float px = t.x > delta ? 1.f : 0.f, nx = t.x < ndelta ? 1.f : 0.f;
                      const float py = t.y > delta ? 1.f : 0.f, ny = t.y < ndelta ? 1.f : 0.f;
                      const float pz = t.z > delta ? 1.f : 0.f, nz = t.z < ndelta ? 1.f : 0.f;
                      const float pw = t.w > delta ? 1.f : 0.f, nw = t.w < ndelta ? 1.f : 0.f;
                      cx += static_cast<double>(fabsf(t.x) * (px + nx));
                      cy += static_cast<double>(fabsf(t.y) * (py + ny));
                      cz += static_cast<double>(fabsf(t.z) * (pz + nz));
                      cw += static_cast<double>(fabsf(t.w) * (pw + nw));
                      byte = pack4({px, nx}, {py, ny}, {pz, nz}, {pw, nw});
                    } else {
                      // the float4 at columns 128q + 4*lane is Philox block (coordinate >> 2)
                      const uint32_t blk = k * (kTile / 4) + r * (kTileCols / 4) + 32 * q + lane;
                      const uint4 x = philox4x32_10(make_uint4(blk, stream_base + m, t_lo, t_hi), key0, key1);
                      const bool kx = philox_uniform(x.x) < __fdiv_rn(fabsf(t.x), scale);
                      const bool ky = philox_uniform(x.y) < __fdiv_rn(fabsf(t.y), scale);
                      const bool kz = philox_uniform(x.z) < __fdiv_rn(fabsf(t.z), scale);
                      const bool kw = philox_uniform(x.w) < __fdiv_rn(fabsf(t.w), scale);
                      byte = pack4(split_code(t.x, kx), split_code(t.y, ky), split_code(t.z, kz), split_code(t.w, kw));
                    }
                    cnt += nonzero_codes(byte);
                  }
                  const uint64_t off = static_cast<uint64_t>(k) * (kTile / 4) + r * (kTileCols / 4) + 32 * q + lane;
                  if (off < row_words * 4) __stcs(codes8 + off, static_cast<uint8_t>(byte));
                }
                return (cx + cy) + (cz + cw);
              });
          return kStochastic ? 0.0 : s;
        }
        LaneCodes lc;
        lc.clear();
        const double s = lane_columns(
            g + static_cast<uint64_t>(m) * geo.ld, tile_base, lane, w, [&](int r, int c, float v) {
              uint32_t code;
              if (!kStochastic) {
                // strict comparisons; a NaN threshold or value compares false and codes 0
                code = v > delta ? 1u : (v < ndelta ? 2u : 0u);
              } else {
                // coordinate i draws word i & 3 of the Philox block i >> 2; |v|/s by IEEE division
                const uint64_t i = tile_base + r * kTileCols + 32 * lane + c;
                const uint4 x = philox4x32_10(make_uint4(static_cast<uint32_t>(i >> 2), stream_base + m, t_lo, t_hi), key0, key1);
                const uint32_t word = (i & 3) == 0 ? x.x : (i & 3) == 1 ? x.y : (i & 3) == 2 ? x.z : x.w;
                const bool keep = philox_uniform(word) < __fdiv_rn(fabsf(v), scale);
                code = keep ? (v > 0.f ? 1u : (v < 0.f ? 2u : 0u)) : 0u;
              }
              cnt += code ? 1u : 0u;
              // the row index is a compile-time constant inside lane_columns' unrolled loops
              if (r == 0) lc.set(0, c, code);
              else if (r == 1) lc.set(1, c, code);
              else if (r == 2) lc.set(2, c, code);
              else lc.set(3, c, code);
              return code ? fabsf(v) : 0.f;
            });
        lc.store(codes + static_cast<uint64_t>(m) * row_words, row_words, k, lane, wide);
        return kStochastic ? 0.0 : warp_pair_tree(s);
      },
      [&](uint32_t m, uint32_t k) {
        LaneCodes lc;
        lc.clear();
        lc.store(codes + static_cast<uint64_t>(m) * row_words, row_words, k, lane, wide);
      },
      [&](uint32_t m, uint32_t c, double picked) {
        const unsigned long long total = block_count(cnt, sm_cnt);
        if (j == 0) {
          const uint64_t p = static_cast<uint64_t>(m) * kMaxChunks + c;
          ws.part_sum[p] = picked;
          ws.part_cnt[p] = total;
        }
      });
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  finish_codes<!kStochastic>(geo, ws, scales_out, counts_out);
  if (j == 0) *ws.ticket = 0u;
}

// As many CTAs as are resident at once (the items differ a lot in cost: no second wave behind a slow one).
template <class Kernel>
unsigned touched_grid(Kernel kernel, const Geometry& geo, const LaunchShape& shape) {
  static int per_sm = 0;  // one instantiation per kernel: asked once (every GPU of a process is the same model)
  if (per_sm < 1 && (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1))
    per_sm = 1;
  const uint64_t items = static_cast<uint64_t>(geo.M) * geo.chunks;
  const uint64_t resident = static_cast<uint64_t>(shape.sm_count) * per_sm;
  return static_cast<unsigned>(items < resident ? items : resident);
}

}  // namespace

int launch_touched_abs_sum(const float* g, const Geometry& geo, float coef, const Workspace& ws, float* thresholds_out,
                           const uint32_t* touched, const LaunchShape& shape, cudaStream_t stream) {
  touched_abs_sum_kernel<<<touched_grid(touched_abs_sum_kernel, geo, shape), kThreads, 0, stream>>>(g, geo, coef, ws, thresholds_out, touched);
  return 1;
}

int launch_touched_abs_max(const float* g, const Geometry& geo, const Workspace& ws, const uint32_t* touched,
                           const LaunchShape& shape, cudaStream_t stream) {
  touched_abs_max_kernel<<<touched_grid(touched_abs_max_kernel, geo, shape), kThreads, 0, stream>>>(g, geo, ws, touched);
  return 1;
}

int launch_touched_codes(bool stochastic, const float* g, const Geometry& geo, uint64_t seed, uint64_t t,
                         const Workspace& ws, uint32_t* codes, float* scales_out, unsigned long long* counts_out,
                         const uint32_t* touched, const LaunchShape& shape, cudaStream_t stream) {
  if (stochastic)
    touched_codes_kernel<true><<<touched_grid(touched_codes_kernel<true>, geo, shape), kThreads, 0, stream>>>(g, geo, seed, t, 0u, ws, codes,
                                                                                 scales_out, counts_out, touched);
  else
    touched_codes_kernel<false><<<touched_grid(touched_codes_kernel<false>, geo, shape), kThreads, 0, stream>>>(g, geo, seed, t, 0u, ws, codes,
                                                                                  scales_out, counts_out, touched);
  return 1;
}

}  // namespace qasg

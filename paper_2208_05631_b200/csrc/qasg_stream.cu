// Passes A and B of the quantizer as ONE launch, for rows that fit the L2 cache.
//
// The threshold Delta_m (Section 3.5) needs the sum over worker m's whole gradient before any of
// its codes can be cut, so a gradient is read twice.  With two kernels (all rows summed, then all rows
// coded) the second read comes from HBM again whenever the M rows together are larger than L2.  Here one
// persistent grid walks the work in the order
//     A(0) T(0) .. A(L-1) T(L-1) | A(L) T(L) B(0) | A(L+1) T(L+1) B(1) | ... | B(M-L) .. B(M-1)
// (A(m) = the sum items of worker m, T(m) = one item that combines their partials into Delta_m and
// publishes it, B(m) = the code items, which wait for T(m)), so a row is coded while it is still in L2,
// L rows after it was summed: the M gradients of a coordinate cross HBM once.  Items are dealt to the
// CTAs round-robin in that order.  The CTA that draws T(m) waits for the last sum items of row m while
// all others go on; with L >= 1 Delta_m has long been published when the code items of row m come up
// (L = 0, for rows too long to keep two in L2, codes row m right behind T(m) and pays that wait).
//
// Forward progress: the launch is cooperative (all CTAs resident), every CTA takes its items in the
// global order, sum items never wait, and a code item waits only for sum items that come earlier in
// that order, so the earliest unfinished item can always run.  Every wait is bounded all the same: after
// max_polls polls the CTA raises kFlagTimeout and the call's abort word, and every CTA returns at its
// next wait (codes of that call are then incomplete and the host learns it from the status word).
//
// Hand-over of the chunk partials: a 64-bit slot per (worker, chunk) that holds kEmptySlot until its item
// has stored its partial there with ONE plain 64-bit store.  The value is the message, so the producer
// needs no fence and no atomic (a fence per item, waiting for the item's own loads in flight, was what
// bounded an earlier form of this kernel); the consumer (T(m), or the CTA that forms the worker's scale at
// the end) polls the slots it needs, takes the values and puts kEmptySlot back, which is also the state the
// next call, or the next replay of a captured launch, expects.
//
// The sums are the fixed-order sums of the two-kernel path (same tiles, same trees): bit-identical results.
#include <type_traits>

#include "qasg_device.cuh"

namespace qasg {

struct StreamItem {
  uint32_t index, kind, m, c, k0, k1;  // kind 0 = sum (A), 1 = codes (B), 2 = combine and publish (T); c = chunk
};

__device__ __forceinline__ uint32_t stream_items_total(const Geometry& geo) { return geo.M * (2u * geo.chunks + 1u); }

__device__ __forceinline__ StreamItem stream_item(const Geometry& geo, uint32_t lag, uint32_t i) {
  const uint32_t ch = geo.chunks;
  StreamItem it;
  it.index = i;
  it.c = 0;
  // stages 0 .. lag-1: A(s) T(s);  stages lag .. M-1: A(s) T(s) B(s - lag);  stages M .. M+lag-1: B(s - lag)
  const uint32_t head = lag * (ch + 1u);
  const uint32_t per = 2u * ch + 1u;
  const uint32_t mid = (geo.M - lag) * per;
  uint32_t q;  // position inside an "A T" block, or ch + 1 + chunk for a code item
  if (i < head) {
    it.m = i / (ch + 1u);
    q = i - it.m * (ch + 1u);
  } else if (i - head < mid) {
    const uint32_t r = i - head, s = r / per;
    q = r - s * per;
    it.m = q <= ch ? lag + s : s;
  } else {
    const uint32_t r = i - head - mid, s = r / ch;
    it.m = geo.M - lag + s;
    q = ch + 1u + (r - s * ch);
  }
  if (q < ch) {
    it.kind = 0;
    it.c = q;
  } else if (q == ch) {
    it.kind = 2;
  } else {
    it.kind = 1;
    it.c = q - ch - 1u;
  }
  it.k0 = it.c * geo.group;
  it.k1 = min(it.k0 + geo.group, geo.tiles);
  return it;
}

// Code bytes of a tile with ordinary (write-back) stores: the codes stay in L2 for pass C.
__device__ __forceinline__ void store_code_bytes_cached(uint8_t* __restrict__ codes8, uint32_t k, int j, bool full,
                                                        uint64_t row_bytes, const uint32_t (&bytes)[kTileRows]) {
  const uint64_t b0 = static_cast<uint64_t>(k) * (kTile / 4) + j;
#pragma unroll
  for (int r = 0; r < kTileRows; ++r)
    if (full || b0 + r * (kTileCols / 4) < row_bytes) codes8[b0 + r * (kTileCols / 4)] = static_cast<uint8_t>(bytes[r]);
}

__device__ __forceinline__ void slot_store(unsigned long long* p, unsigned long long v) {
  asm volatile("st.relaxed.gpu.global.u64 [%0], %1;" ::"l"(p), "l"(v) : "memory");
}
__device__ __forceinline__ unsigned long long slot_load(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.relaxed.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p));
  return v;
}

// Waits, within the bound, until the slot holds a value, and returns it.  ok is cleared if the wait ran out.
__device__ __noinline__ unsigned long long slot_wait(const unsigned long long* p, unsigned int* abort_word,
                                                     unsigned int* status, uint32_t max_polls, bool& ok) {
  for (uint32_t i = 0; i < max_polls; ++i) {
    const unsigned long long v = slot_load(p);
    if (v != kEmptySlot) return v;
    if (load_relaxed(abort_word) != 0u) break;
    __nanosleep(i < 32 ? 20 : 200);
  }
  atomicExch(abort_word, 1u);
  atomicOr(status, kFlagTimeout);
  ok = false;
  return 0ull;
}

// Takes eight adjacent slots (those at or past `count` read as 0): all eight loads go out together, a slot
// found empty is then waited for on its own, and the taken slots are left empty.
__device__ __forceinline__ void slots_take8(unsigned long long* p, uint32_t first, uint32_t count,
                                            unsigned int* abort_word, unsigned int* status, uint32_t max_polls,
                                            bool& ok, unsigned long long (&v)[8]) {
#pragma unroll
  for (int k = 0; k < 8; ++k) v[k] = first + k < count ? slot_load(p + first + k) : 0ull;
#pragma unroll
  for (int k = 0; k < 8; ++k)
    if (v[k] == kEmptySlot) v[k] = slot_wait(p + first + k, abort_word, status, max_polls, ok);
#pragma unroll
  for (int k = 0; k < 8; ++k)
    if (first + k < count) slot_store(p + first + k, kEmptySlot);
}

// warp_chunk_tree over slots that are taken (and emptied) on the way: the same additions in the same order.
__device__ __forceinline__ double warp_slot_tree(unsigned long long* slots, uint32_t chunks, int lane,
                                                 unsigned int* abort_word, unsigned int* status, uint32_t max_polls,
                                                 bool& ok) {
  double top[4];
#pragma unroll 1
  for (int q = 0; q < 4; ++q) {
    unsigned long long bits[8];
    slots_take8(slots, lane * 32 + q * 8, chunks, abort_word, status, max_polls, ok, bits);
    double v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = __longlong_as_double(static_cast<long long>(bits[k]));
    top[q] = ((v[0] + v[1]) + (v[2] + v[3])) + ((v[4] + v[5]) + (v[6] + v[7]));
  }
  return warp_pair_tree((top[0] + top[1]) + (top[2] + top[3]));
}

// Order-free reductions over a worker's slots (sum of counts, maximum), taken the same way.
template <bool kMax>
__device__ __forceinline__ unsigned long long warp_slot_reduce(unsigned long long* slots, uint32_t chunks, int lane,
                                                               unsigned int* abort_word, unsigned int* status,
                                                               uint32_t max_polls, bool& ok) {
  unsigned long long acc = 0ull;
#pragma unroll 1
  for (int q = 0; q < 4; ++q) {
    unsigned long long bits[8];
    slots_take8(slots, lane * 32 + q * 8, chunks, abort_word, status, max_polls, ok, bits);
#pragma unroll
    for (int k = 0; k < 8; ++k) acc = kMax ? (bits[k] > acc ? bits[k] : acc) : acc + bits[k];
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    const unsigned long long o = __shfl_xor_sync(0xffffffffu, acc, s);
    acc = kMax ? (o > acc ? o : acc) : acc + o;
  }
  return acc;
}

// The fixed-order sum of an item's tiles (the arithmetic of ChunkSum, tile by tile the same additions)
// with the item's count of kept coordinates carried through the same two CTA-wide meetings, so that an
// item ends with one flush and nothing else.  An item is at most kItemTiles tiles long.
constexpr int kItemTiles = 32;
struct ItemSumStorage {
  double warp_sums[kItemTiles][kThreads / 32];
  double tile_sums[kItemTiles];
  // Written before an item's flush and read after it, by threads that do not meet again until the next
  // flush: two copies, used by alternate items, keep an early writer away from a late reader.
  uint32_t warp_cnts[2][kThreads / 32];
  uint32_t ready[2];  // thread 0's look at the next item's "published" word, handed to the CTA across the flush
};

// Item T(m): the worker's threshold (or scaler) from the chunk partials of its sum items, taken out of
// their slots by one warp.  All threads of the CTA call; the statistic is published when it returns true.
// Kept out of line: it runs once per worker and must not weigh on the registers of the tile loop.
template <bool kStochastic>
__device__ __noinline__ bool stream_publish_level(uint32_t m, uint32_t chunks, uint64_t d, float coef, uint32_t max_polls,
                                                  const Workspace& ws, const StreamSlots& slots, StreamSync* sync,
                                                  float* thresholds_out, bool* sm_flag) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (warp == 0) {
    bool ok = true;
    unsigned long long* mine = slots.sum_a + static_cast<uint64_t>(m) * kMaxChunks;
    float stat;
    bool nonfinite;
    if (kStochastic) {
      const uint32_t bmax =
          static_cast<uint32_t>(warp_slot_reduce<true>(mine, chunks, lane, &sync->abort, ws.status, max_polls, ok));
      stat = __uint_as_float(bmax);
      nonfinite = bmax >= 0x7f800000u;
    } else {
      const double s = warp_slot_tree(mine, chunks, lane, &sync->abort, ws.status, max_polls, ok);
      stat = static_cast<float>((static_cast<double>(coef) * s) / static_cast<double>(d));
      nonfinite = !isfinite(s);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (lane == 0) {
      if (ok) {
        if (kStochastic) ws.scales[m] = stat;
        ws.thresholds[m] = kStochastic ? 0.f : stat;
        if (thresholds_out) thresholds_out[m] = kStochastic ? 0.f : stat;
        if (nonfinite) atomicOr(ws.status, kFlagNonFinite);
        __threadfence();
        store_release(&sync->ready[m], 1u);
      }
      *sm_flag = ok;
    }
  }
  __syncthreads();
  return *sm_flag;
}

// The scale and count of worker m once all its code items are in (one warp).
template <bool kStochastic>
__device__ __noinline__ void stream_publish_scale(uint32_t m, uint32_t chunks, uint32_t max_polls, const Workspace& ws,
                                                  const StreamSlots& slots, StreamSync* sync, float* scales_out,
                                                  unsigned long long* counts_out) {
  const int lane = threadIdx.x & 31;
  bool ok = true;
  const unsigned long long n = warp_slot_reduce<false>(slots.cnt_b + static_cast<uint64_t>(m) * kMaxChunks, chunks, lane,
                                                       &sync->abort, ws.status, max_polls, ok);
  float scale;
  if (kStochastic) {
    scale = __ldcg(ws.scales + m);
  } else {
    const double p = warp_slot_tree(slots.sum_b + static_cast<uint64_t>(m) * kMaxChunks, chunks, lane, &sync->abort,
                                    ws.status, max_polls, ok);
    scale = n ? static_cast<float>(p / static_cast<double>(n)) : 0.f;
  }
  ok = __all_sync(0xffffffffu, ok);
  if (ok && lane == 0) {
    ws.counts[m] = n;
    if (!kStochastic) ws.scales[m] = scale;
    if (scales_out) scales_out[m] = scale;
    if (counts_out) counts_out[m] = n;
    sync->ready[m] = 0u;  // every code item of the worker has passed its wait: as the next call expects it
  }
}

// kStochastic: A takes max|g| (the scaler), B draws Philox codes; else A sums |g| (Delta), B cuts Q_Delta.
// kKeepCodes: the code bytes are written with ordinary stores (kept in L2), else with streaming stores.
//
// Shape of the code: the walk over a CTA's items is the outer loop; an item's tiles are walked by a tight
// inner loop specialised for its kind (two tiles per turn, the next tile's loads always in flight, the
// first tile of the CTA's next item requested during the item's last tile).  What is needed only between
// items (decoding an index, the combine duty, the waits) stays out of that loop and out of its registers.
template <bool kStochastic, bool kKeepCodes>
__global__ void __launch_bounds__(kThreads, 4)
quantize_stream_kernel(const float* __restrict__ g, Geometry geo, StreamParams sp, Workspace ws, StreamSlots slots,
                       StreamSync* sync, uint32_t* __restrict__ codes, float* __restrict__ scales_out,
                       float* __restrict__ thresholds_out, unsigned long long* __restrict__ counts_out) {
  __shared__ ItemSumStorage sm;
  __shared__ bool sm_flag;
  const int j = threadIdx.x, warp = j >> 5, lane = j & 31;
  const uint32_t total = stream_items_total(geo);
  if (blockIdx.x >= total) return;

  // A call that gave up leaves slots and words in an unknown state: until the host has cleared them
  // (qasg_last_async_status does, when it reports the time-out) no further call does anything.
  if (j == 0) {
    sm_flag = load_relaxed(&sync->abort) == 0u;
    if (!sm_flag) atomicOr(ws.status, kFlagTimeout);
  }
  __syncthreads();
  if (!sm_flag) return;

  uint32_t par = 0u;
  float4 a[kTileRows], b[kTileRows];

  // Finds the CTA's next item with tiles at index `from`.  A combine item there is not done yet (the item in
  // hand must end first): its worker goes to `duty`, the index behind it to `resume`; resume = total when the
  // CTA's items are exhausted.
  constexpr uint32_t kNoDuty = 0xFFFFFFFFu;
  uint32_t duty = kNoDuty, resume = total;
  auto scan = [&](uint32_t from, StreamItem& out) -> bool {
    duty = kNoDuty;
    resume = total;
    if (from >= total) return false;
    out = stream_item(geo, sp.lag, from);
    if (out.kind != 2u) return true;
    duty = out.m;
    resume = from + gridDim.x;
    return false;
  };

  // The tiles of one item.  On entry the item's first tile is in `a`; on return `a` holds the first tile of
  // `nxt` (the CTA's next item with tiles) if has_next.  Returns thread 0's early look at nxt's "published" word.
  auto run_item = [&](auto kind_tag, const StreamItem& cur, float level, StreamItem& nxt, bool& has_next,
                      uint32_t& cnt_out, uint32_t& pending_out) -> uint32_t {
    constexpr bool kCodes = decltype(kind_tag)::value;
    const float* __restrict__ row = g + static_cast<uint64_t>(cur.m) * geo.ld;
    const uint64_t row_words = (geo.d + 15) >> 4;
    uint8_t* codes8 = reinterpret_cast<uint8_t*>(codes + static_cast<uint64_t>(cur.m) * row_words);
    const uint32_t full_tiles = static_cast<uint32_t>(geo.d / kTile);
    const uint32_t k1 = cur.k1;
    uint32_t k = cur.k0, pending = 0u, acc = 0u, next_ready = 0u;

    auto process = [&](const float4 (&v)[kTileRows], uint32_t kk) {
      if (!kCodes) {
        if (kStochastic) {
#pragma unroll
          for (int r = 0; r < kTileRows; ++r) {
            acc = max(acc, __float_as_uint(fabsf(v[r].x)));
            acc = max(acc, __float_as_uint(fabsf(v[r].y)));
            acc = max(acc, __float_as_uint(fabsf(v[r].z)));
            acc = max(acc, __float_as_uint(fabsf(v[r].w)));
          }
        } else {
          double cx = fabsf(v[0].x), cy = fabsf(v[0].y), cz = fabsf(v[0].z), cw = fabsf(v[0].w);
#pragma unroll
          for (int r = 1; r < kTileRows; ++r) {
            cx += static_cast<double>(fabsf(v[r].x));
            cy += static_cast<double>(fabsf(v[r].y));
            cz += static_cast<double>(fabsf(v[r].z));
            cw += static_cast<double>(fabsf(v[r].w));
          }
          const double w = warp_pair_tree((cx + cy) + (cz + cw));
          if (lane == 0) sm.warp_sums[pending][warp] = w;
          ++pending;
        }
        return;
      }
      uint32_t bytes[kTileRows];
      if (kStochastic) {
        const uint32_t key0 = static_cast<uint32_t>(sp.seed), key1 = static_cast<uint32_t>(sp.seed >> 32);
        const uint32_t t_lo = static_cast<uint32_t>(sp.t), t_hi = static_cast<uint32_t>(sp.t >> 32);
#pragma unroll
        for (int r = 0; r < kTileRows; ++r) {
          const float4 t = v[r];
          const uint32_t blk = kk * (kTile / 4) + r * (kTileCols / 4) + j;
          const uint4 w = philox4x32_10(make_uint4(blk, sp.stream_base + cur.m, t_lo, t_hi), key0, key1);
          const bool kx = philox_uniform(w.x) < __fdiv_rn(fabsf(t.x), level);
          const bool ky = philox_uniform(w.y) < __fdiv_rn(fabsf(t.y), level);
          const bool kz = philox_uniform(w.z) < __fdiv_rn(fabsf(t.z), level);
          const bool kw = philox_uniform(w.w) < __fdiv_rn(fabsf(t.w), level);
          bytes[r] = pack4(split_code(t.x, kx), split_code(t.y, ky), split_code(t.z, kz), split_code(t.w, kw));
          acc += nonzero_codes(bytes[r]);
        }
      } else {
        const float nlevel = -level;
        double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
        float cntf = 0.f;
#pragma unroll
        for (int r = 0; r < kTileRows; ++r) {
          const float4 t = v[r];
          const float px = t.x > level ? 1.f : 0.f, nx = t.x < nlevel ? 1.f : 0.f;
          const float py = t.y > level ? 1.f : 0.f, ny = t.y < nlevel ? 1.f : 0.f;
          const float pz = t.z > level ? 1.f : 0.f, nz = t.z < nlevel ? 1.f : 0.f;
          const float pw = t.w > level ? 1.f : 0.f, nw = t.w < nlevel ? 1.f : 0.f;
          const float kx = px + nx, ky = py + ny, kz = pz + nz, kw = pw + nw;
          cx += static_cast<double>(fabsf(t.x) * kx);
          cy += static_cast<double>(fabsf(t.y) * ky);
          cz += static_cast<double>(fabsf(t.z) * kz);
          cw += static_cast<double>(fabsf(t.w) * kw);
          cntf += (kx + ky) + (kz + kw);
          bytes[r] = pack4({px, nx}, {py, ny}, {pz, nz}, {pw, nw});
        }
        acc += static_cast<uint32_t>(cntf);
        const double w = warp_pair_tree((cx + cy) + (cz + cw));
        if (lane == 0) sm.warp_sums[pending][warp] = w;
        ++pending;
      }
      if (kKeepCodes)
        store_code_bytes_cached(codes8, kk, j, kk < full_tiles, row_words * 4, bytes);
      else
        store_code_bytes(codes8, kk, j, kk < full_tiles, row_words * 4, bytes);
    };
    // All tiles but the last: the tile in hand and the one requested both belong to this item, and nothing
    // that concerns other items is touched (or kept in registers) here.
    while (k + 2 < k1) {
      load_tile(row, static_cast<uint64_t>(k + 1) * kTile, geo.d, j, b);
      process(a, k);
      load_tile(row, static_cast<uint64_t>(k + 2) * kTile, geo.d, j, a);
      process(b, k + 1);
      k += 2;
    }
    if (k + 2 == k1) {
      load_tile(row, static_cast<uint64_t>(k + 1) * kTile, geo.d, j, b);
      process(a, k);
      ++k;
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) a[r] = b[r];
    }
    // The last tile: while it is processed, the first tile of the CTA's next item is requested, and thread 0
    // looks at that item's "published" word; both answers are back by the time they are needed.  The scan
    // stops at a combine item: that duty comes after this item has ended, and the item behind it is then
    // loaded without overlap.
    has_next = scan(cur.index + gridDim.x, nxt);
    if (has_next) {
      load_tile(g + static_cast<uint64_t>(nxt.m) * geo.ld, static_cast<uint64_t>(nxt.k0) * kTile, geo.d, j, b);
      if (nxt.kind == 1u && j == 0) next_ready = load_acquire(&sync->ready[nxt.m]);
    }
    process(a, k);
    if (has_next) {
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) a[r] = b[r];
    }
    cnt_out = acc;
    pending_out = pending;
    return next_ready;
  };

  // After the last tile of an item: one flush (two CTA-wide meetings) turns the parked warp sums into the
  // chunk's fixed-order sum, carries the count (or the maximum) along, and hands `next_ready` (known to
  // thread 0 only) to every thread.  Thread 0 then stores the chunk's partial into its slot.
  auto end_item = [&](const StreamItem& it, uint32_t acc, uint32_t pending, uint32_t next_ready) -> bool {
    const uint64_t slot = static_cast<uint64_t>(it.m) * kMaxChunks + it.c;
    const bool is_max = kStochastic && it.kind == 0u;
    const uint32_t wred = is_max ? __reduce_max_sync(0xffffffffu, acc) : __reduce_add_sync(0xffffffffu, acc);
    par ^= 1u;
    if (lane == 0) sm.warp_cnts[par][warp] = wred;
    if (j == 0) sm.ready[par] = next_ready;
    __syncthreads();
    if (!kStochastic && static_cast<uint32_t>(j) < pending) {
      const double* w = sm.warp_sums[j];
      sm.tile_sums[j] = ((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]));
    }
    __syncthreads();
    const bool ready = sm.ready[par] != 0u;
    if (j == 0) {
      double chunk_total = 0.0;
      if (!kStochastic) {
        double stack[8];  // pairwise tree over the item's tiles (at most kItemTiles = 2^5 of them)
        for (uint32_t i = 0; i < pending; ++i) tile_push(stack, i, sm.tile_sums[i]);
        chunk_total = tile_fold(stack, pending, geo.log2_group);
      }
      uint32_t red = sm.warp_cnts[par][0];
#pragma unroll
      for (int w = 1; w < kThreads / 32; ++w) red = is_max ? max(red, sm.warp_cnts[par][w]) : red + sm.warp_cnts[par][w];
      const unsigned long long total_bits = static_cast<unsigned long long>(__double_as_longlong(chunk_total));
      if (it.kind == 0u) {
        slot_store(slots.sum_a + slot, kStochastic ? static_cast<unsigned long long>(red) : total_bits);
      } else {
        if (!kStochastic) slot_store(slots.sum_b + slot, total_bits);
        slot_store(slots.cnt_b + slot, static_cast<unsigned long long>(red));
      }
    }
    return ready;
  };

  StreamItem cur, nxt;
  uint32_t from = blockIdx.x;
  bool have = false, ready = false, alive = true;
  for (;;) {
    if (!have) {  // at the start, and behind a combine item: nothing is in flight
      if (duty != kNoDuty &&  // the combine item the last scan stopped at: now is its turn
          !stream_publish_level<kStochastic>(duty, geo.chunks, geo.d, sp.coef, sp.max_polls, ws, slots, sync,
                                             thresholds_out, &sm_flag)) {
        alive = false;
        break;
      }
      have = scan(from, cur);
      if (!have) {
        if (duty == kNoDuty) break;  // the CTA's items are exhausted
        from = resume;
        continue;
      }
      load_tile(g + static_cast<uint64_t>(cur.m) * geo.ld, static_cast<uint64_t>(cur.k0) * kTile, geo.d, j, a);
      ready = false;
    }
    float level = 0.f;
    if (cur.kind == 1u) {  // a code item needs its worker's threshold (or scaler)
      if (!ready) {
        if (j == 0) sm_flag = wait_for_value(&sync->ready[cur.m], 1u, &sync->abort, ws.status, sp.max_polls);
        __syncthreads();
        if (!sm_flag) {
          alive = false;
          break;
        }
      }
      level = kStochastic ? __ldcg(ws.scales + cur.m) : __ldcg(ws.thresholds + cur.m);
    }
    bool has_next = false;
    uint32_t acc = 0u, pending = 0u, next_ready;
    if (cur.kind == 0u)
      next_ready = run_item(std::false_type{}, cur, level, nxt, has_next, acc, pending);
    else
      next_ready = run_item(std::true_type{}, cur, level, nxt, has_next, acc, pending);
    ready = end_item(cur, acc, pending, next_ready);
    have = has_next;
    if (has_next) {
      cur = nxt;
    } else {
      from = resume;  // behind the combine item the scan stopped at, or past the end
    }
  }
  // The scale and count of worker m = blockIdx.x once all its code items are in.  Every wait above was for
  // an item earlier in the order; this one is for items that other CTAs finish without waiting for us.
  if (alive && blockIdx.x < geo.M && warp == 0)
    stream_publish_scale<kStochastic>(blockIdx.x, geo.chunks, sp.max_polls, ws, slots, sync, scales_out, counts_out);
}

// Waits that nothing ends: both bounded waits (for a value; for a counter to reach a target) on a word that
// no one sets.  The kernel returns after 2 * max_polls polls with kFlagTimeout raised, only if both waits
// gave up; nothing else is touched.
__global__ void wait_selftest_kernel(StreamSync* sync, unsigned int* status, uint32_t max_polls) {
  __shared__ unsigned int local_status;  // the waits raise their flag with an atomic: shared, not local, memory
  if (threadIdx.x == 0) {
    local_status = 0u;
    sync->probe_abort = 0u;
    const bool a = wait_for_value(&sync->probe, 0xFFFFFFFFu, &sync->probe_abort, &local_status, max_polls);
    sync->probe_abort = 0u;
    const bool b = wait_until_at_least(&sync->probe, 1u, &sync->probe_abort, &local_status, max_polls);
    if (!a && !b && local_status == kFlagTimeout) atomicOr(status, kFlagTimeout);
  }
}

namespace {
template <bool kStochastic, bool kKeepCodes>
cudaError_t launch_stream_as(const float* g, const Geometry& geo, const StreamParams& sp, const Workspace& ws,
                             const StreamSlots& slots, StreamSync* sync, uint32_t* codes, float* scales_out, float* thresholds_out,
                             unsigned long long* counts_out, const LaunchShape& shape, cudaStream_t stream) {
  auto kernel = quantize_stream_kernel<kStochastic, kKeepCodes>;
  static thread_local int ctas_per_sm[64] = {0};  // per device, resolved on first use
  int dev = 0;
  cudaGetDevice(&dev);
  int& resident = ctas_per_sm[dev & 63];
  if (resident == 0) {
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kThreads, 0);
    if (resident < 1) resident = 1;
  }
  const uint64_t total = static_cast<uint64_t>(geo.M) * (2ull * geo.chunks + 1);
  const uint64_t capacity = static_cast<uint64_t>(shape.sm_count) * resident;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(total < capacity ? total : capacity));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;  // all CTAs resident together: the waits between them end
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, g, geo, sp, ws, slots, sync, codes, scales_out, thresholds_out, counts_out);
}
}  // namespace

int launch_quantize_stream(bool stochastic, bool keep_codes, const float* g, const Geometry& geo,
                           const StreamParams& sp, const Workspace& ws, const StreamSlots& slots, StreamSync* sync,
                           uint32_t* codes,
                           float* scales_out, float* thresholds_out, unsigned long long* counts_out,
                           const LaunchShape& shape, cudaStream_t stream) {
  if (stochastic) {
    if (keep_codes)
      launch_stream_as<true, true>(g, geo, sp, ws, slots, sync, codes, scales_out, thresholds_out, counts_out, shape,
                                   stream);
    else
      launch_stream_as<true, false>(g, geo, sp, ws, slots, sync, codes, scales_out, thresholds_out, counts_out, shape,
                                   stream);
  } else {
    if (keep_codes)
      launch_stream_as<false, true>(g, geo, sp, ws, slots, sync, codes, scales_out, thresholds_out, counts_out, shape,
                                   stream);
    else
      launch_stream_as<false, false>(g, geo, sp, ws, slots, sync, codes, scales_out, thresholds_out, counts_out, shape,
                                   stream);
  }
  return 1;
}

int launch_wait_selftest(StreamSync* sync, unsigned int* status, uint32_t max_polls, cudaStream_t stream) {
  wait_selftest_kernel<<<1, 32, 0, stream>>>(sync, status, max_polls);
  return 1;
}

}  // namespace qasg

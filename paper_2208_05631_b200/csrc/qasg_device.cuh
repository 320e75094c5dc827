// Device-side building blocks shared by the kernel files: tile loads, the fixed-order sums,
// the grid-completion ticket, the stream of tiles of a CTA, code-byte packing, Philox4x32-10.
#pragma once
#include "qasg_internal.h"

namespace qasg {

// ------------------------------------------------------------------ chained launches
// Programmatic dependent launch: a kernel launched with the attribute below may start while its predecessor
// in the stream is still running (once every CTA of the predecessor has passed chain_trigger or exited).  The
// rules every chained kernel here keeps:
//   - chain_wait() comes before the first access to anything a predecessor may have written; it returns once
//     the predecessor grid has completed and its writes are visible;
//   - chain_trigger() comes after chain_wait(), so when a dependent starts, everything older than its
//     immediate predecessor is complete: a dependent may therefore read, ahead of its own chain_wait(),
//     only data that its immediate predecessor does not write (the gradients, in pass B).
// Both are no-ops in a kernel launched without the attribute.
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), unsigned grid, unsigned block, size_t smem,
                                  cudaStream_t stream, bool chained, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ------------------------------------------------------------------ device helpers
__device__ __forceinline__ float4 load_f4(const float* p) {
  return __ldg(reinterpret_cast<const float4*>(p));
}

// The four float4 a thread owns in the tile starting at coordinate tile_base.
// Coordinates >= d read as +0.0 (they neither count nor code).
__device__ __forceinline__ void load_tile(const float* __restrict__ row, uint64_t tile_base,
                                          uint64_t d, int j, float4 (&v)[kTileRows]) {
  if (tile_base + kTile <= d) {
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) v[r] = load_f4(row + tile_base + r * kTileCols + 4 * j);
  } else {
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      const uint64_t i0 = tile_base + r * kTileCols + 4 * j;
      float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
      if (i0 < d) {
        t = load_f4(row + i0);  // stays inside the row: ld is a multiple of 4 and >= d
        if (i0 + 1 >= d) t.y = 0.f;
        if (i0 + 2 >= d) t.z = 0.f;
        if (i0 + 3 >= d) t.w = 0.f;
      }
      v[r] = t;
    }
  }
}

// Pairwise tree over the 32 lanes (adjacent pairs first).  Addition commutes bit for bit,
// so both partners of every exchange hold the same value.
__device__ __forceinline__ double warp_pair_tree(double v) {
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) v += __shfl_xor_sync(0xffffffffu, v, s);
  return v;
}

// Streaming pairwise summation over the tiles of a chunk (thread 0 only): stack[l] holds
// the sum of a complete aligned subtree of 2^l tiles.
__device__ __forceinline__ void tile_push(double* stack, uint32_t k_local, double v) {
  int lvl = 0;
  while (k_local & 1u) {
    v = stack[lvl] + v;
    k_local >>= 1;
    ++lvl;
  }
  stack[lvl] = v;
}
// Completes the chunk's tree after n <= 2^log2_group tiles (missing tiles are +0.0).
__device__ __forceinline__ double tile_fold(const double* stack, uint32_t n, uint32_t log2_group) {
  double carry = 0.0;
  for (uint32_t lvl = 0; lvl <= log2_group; ++lvl)
    if ((n >> lvl) & 1u) carry = stack[lvl] + carry;
  return carry;
}

// Fixed-order sum over the tiles of one chunk.  Every tile, each thread contributes the sum
// of its 4 columns; the warp butterfly runs at once, but the eight warp sums of a tile are only
// parked in shared memory.  Every kBatchTiles tiles (and at the end of the chunk) the CTA meets
// once: the parked sums are combined tile by tile (pairwise over the 8 warps), then pushed, in
// tile order, onto the chunk's pairwise stack.  The order of additions is the same as if every
// tile had been reduced on its own; the warps just do not wait for each other at every tile.
constexpr int kBatchTiles = 64;
struct ChunkSumStorage {
  double warp_sums[kBatchTiles][kThreads / 32];
  double tile_sums[kBatchTiles];
  double stack[32];
};

class ChunkSum {
 public:
  __device__ __forceinline__ ChunkSum(ChunkSumStorage* st) : st_(st), pending_(0), pushed_(0) {}

  // Called by all threads, once per tile, in tile order.
  __device__ __forceinline__ void add_tile(double thread_sum) { add_warp_sum(warp_pair_tree(thread_sum)); }

  // The same with the warp's butterfly already taken (or skipped: a warp of zeros sums to +0.0).
  __device__ __forceinline__ void add_warp_sum(double v) {
    if ((threadIdx.x & 31) == 0) st_->warp_sums[pending_][threadIdx.x >> 5] = v;
    if (++pending_ == kBatchTiles) flush();
  }

  // Called by all threads after the chunk's last tile; the chunk sum is valid in thread 0.
  __device__ __forceinline__ double finish(uint32_t log2_group) {
    if (pending_) flush();
    double r = 0.0;
    if (threadIdx.x == 0) r = tile_fold(st_->stack, pushed_, log2_group);
    pushed_ = 0;
    return r;
  }

 private:
  __device__ __forceinline__ void flush() {
    __syncthreads();
    if (threadIdx.x < pending_) {
      const double* a = st_->warp_sums[threadIdx.x];
      st_->tile_sums[threadIdx.x] = ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
    }
    __syncthreads();
    if (threadIdx.x == 0)
      for (uint32_t i = 0; i < pending_; ++i) tile_push(st_->stack, pushed_ + i, st_->tile_sums[i]);
    pushed_ += pending_;
    pending_ = 0;
  }
  ChunkSumStorage* st_;
  uint32_t pending_, pushed_;
};

// Pairwise tree over a worker's kMaxChunks partial slots (slots >= chunks are +0.0),
// computed by one warp: 32 adjacent slots per lane, then the lane butterfly.
// kRounds: in how many rounds the lane's 32 slots are requested (4: eight at a time, few registers; 1: all
// before the first is used, one round trip to L2 instead of four).  The sum is the same.
template <int kRounds = 4>
__device__ __forceinline__ double warp_chunk_tree(const double* part, uint32_t chunks, int lane) {
  constexpr int kPer = 32 / kRounds;  // slots per round
  double top[4];
#pragma unroll 1
  for (int q0 = 0; q0 < 4; q0 += 4 / kRounds) {
    double v[kPer];
#pragma unroll
    for (int k = 0; k < kPer; ++k) {
      const uint32_t idx = lane * 32 + q0 * 8 + k;
      v[k] = idx < chunks ? __ldcg(part + idx) : 0.0;
    }
#pragma unroll
    for (int q = 0; q < 4 / kRounds; ++q)
      top[q0 + q] = ((v[8 * q] + v[8 * q + 1]) + (v[8 * q + 2] + v[8 * q + 3])) +
                    ((v[8 * q + 4] + v[8 * q + 5]) + (v[8 * q + 6] + v[8 * q + 7]));
  }
  return warp_pair_tree((top[0] + top[1]) + (top[2] + top[3]));
}

// True in every thread of the CTA that finishes last.  All global writes this CTA made
// before the call (by thread 0) are visible to that CTA.
__device__ __forceinline__ bool grid_last_cta(unsigned int* ticket, bool* sm_flag) {
  if (threadIdx.x == 0) {
    __threadfence();
    const unsigned int prev = atomicAdd(ticket, 1u);
    *sm_flag = (prev == gridDim.x - 1);
  }
  __syncthreads();
  const bool last = *sm_flag;
  if (last) __threadfence();
  return last;
}

// ------------------------------------------------------------------ waits between CTAs (always bounded)
__device__ __forceinline__ unsigned int load_acquire(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void store_release(unsigned int* p, unsigned int v) {
  asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
__device__ __forceinline__ unsigned int load_relaxed(const unsigned int* p) {
  unsigned int v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}

// One thread polls *flag until it holds `value`.  Gives up after max_polls polls (raising the abort
// word and kFlagTimeout) or as soon as another CTA has given up.
__device__ __forceinline__ bool wait_for_value(const unsigned int* flag, unsigned int value, unsigned int* abort_word,
                                            unsigned int* status, uint32_t max_polls) {
  for (uint32_t i = 0; i < max_polls; ++i) {
    if (load_acquire(flag) == value) return true;
    if (load_relaxed(abort_word) != 0u) break;
    __nanosleep(i < 32 ? 20 : 200);
  }
  atomicExch(abort_word, 1u);
  atomicOr(status, kFlagTimeout);
  return false;
}

// One thread polls *counter until it holds at least `target` (a counter that only grows during the launch).
__device__ __forceinline__ bool wait_until_at_least(const unsigned int* counter, unsigned int target,
                                                    unsigned int* abort_word, unsigned int* status, uint32_t max_polls) {
  for (uint32_t i = 0; i < max_polls; ++i) {
    const unsigned int gave_up = load_relaxed(abort_word);  // both loads are in flight together
    const unsigned int arrived = load_acquire(counter);
    if (gave_up != 0u) break;  // first: after a launch that gave up the counter means nothing
    if (arrived >= target) return true;
    if (i >= 64) __nanosleep(i < 1024 ? 40 : 400);
  }
  atomicExch(abort_word, 1u);
  atomicOr(status, kFlagTimeout);
  return false;
}

// All CTAs of a launch whose CTAs are resident together (a cooperative launch, or a single CTA) meet for the
// `phase`-th time (1, 2, ...), and combine() (all threads of a CTA; it reads what the CTAs wrote to global
// memory before they arrived and writes the same values whichever CTA runs it) has run before anyone goes on:
//  * up to kMeetEveryone CTAs: everyone waits until all have arrived and then runs combine() itself (the
//    shortest chain of round trips through L2);
//  * more CTAs: the one that arrives last runs it and lets the others go (hundreds of CTAs reading the same
//    few lines at once cost more than the extra hand-over).
// What combine() wrote is visible to every thread of every CTA after the call (read it with loads that do
// not go through L1 lines filled earlier in the launch).  Returns false in every thread of the CTA if the
// wait ran out.
// kLast: this is the launch's last meeting.  A CTA that has passed it says so; the one that says so last knows
// that no CTA looks at the words any more and puts them back to zero for the next launch.
// After a launch that gave up (the abort word is set until the host has cleared the words) every wait fails at
// once: no further launch gets past its first meeting.
constexpr unsigned int kMeetEveryone = 160;
template <bool kLast, class Combine>
__device__ __forceinline__ bool grid_meet(StreamSync* sync, uint32_t phase, uint32_t max_polls, unsigned int* status,
                                          uint32_t* sm_word, Combine&& combine) {
  __threadfence();
  __syncthreads();
  if (gridDim.x == 1) {
    combine();
    __syncthreads();
    return true;
  }
  bool ok;
  if (gridDim.x <= kMeetEveryone) {
    if (threadIdx.x == 0) {
      atomicAdd(&sync->meet_count, 1u);
      *sm_word = wait_until_at_least(&sync->meet_count, phase * gridDim.x, &sync->abort, status, max_polls) ? 1u : 0u;
    }
    __syncthreads();
    ok = *sm_word != 0u;
    if (ok) combine();
    __syncthreads();
  } else {
    if (threadIdx.x == 0) *sm_word = atomicAdd(&sync->meet_count, 1u) == phase * gridDim.x - 1 ? 1u : 0u;
    __syncthreads();
    const bool last = *sm_word != 0u;
    if (last) {
      __threadfence();
      combine();
      __threadfence();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      if (last) {
        store_release(&sync->meet_go, phase);
        *sm_word = 1u;
      } else {
        *sm_word = wait_until_at_least(&sync->meet_go, phase, &sync->abort, status, max_polls) ? 1u : 0u;
      }
    }
    __syncthreads();
    ok = *sm_word != 0u;
  }
  // said by a thread that the work right behind the meeting does not wait for
  if (kLast && ok && threadIdx.x == blockDim.x - 1) {
    if (atomicAdd(&sync->meet_exit, 1u) == gridDim.x - 1) {
      sync->meet_count = 0u;
      sync->meet_go = 0u;
      sync->meet_exit = 0u;
    }
  }
  return ok;
}

// Calls body(tile_values, k) for the tiles k0 <= k < k1 of one worker row, keeping the loads
// of tile k+1 in flight while tile k is processed (two register buffers, no copies).
template <class Body>
__device__ __forceinline__ void walk_tiles(const float* __restrict__ row, uint64_t d, uint32_t k0,
                                           uint32_t k1, int j, Body&& body) {
  float4 a[kTileRows], b[kTileRows];
  load_tile(row, static_cast<uint64_t>(k0) * kTile, d, j, a);
  uint32_t k = k0;
  while (true) {
    if (k + 1 < k1) load_tile(row, static_cast<uint64_t>(k + 1) * kTile, d, j, b);
    body(a, k);
    if (++k >= k1) break;
    if (k + 1 < k1) load_tile(row, static_cast<uint64_t>(k + 1) * kTile, d, j, a);
    body(b, k);
    if (++k >= k1) break;
  }
}

// The indicator bits of tile k as a warp needs them (its 128 columns of the 4 rows = 16 words): lane
// l < 16 holds the word of row l>>2, quarter l&3, the other lanes 0; a thread's nibble of row r comes
// out of the holder's word by one shuffle (all lanes of the warp must call nibble together).
struct TileMask {
  uint32_t word;
  __device__ __forceinline__ uint32_t nibble(int r, int j) const {
    const int lane = j & 31;
    const uint32_t w = __shfl_sync(0xffffffffu, word, r * 4 + (lane >> 3));
    return (w >> (4 * (lane & 7))) & 15u;
  }
};
// words: the worker's row of indicator words (bits at or past d are 0 there).
__device__ __forceinline__ void load_tile_mask(const uint32_t* __restrict__ words, uint64_t d, uint32_t k, int j,
                                               TileMask& mask) {
  const int lane = j & 31, warp = j >> 5;
  const uint64_t idx = static_cast<uint64_t>(k) * (kTile / 32) + (lane >> 2) * (kTileCols / 32) + 4 * warp + (lane & 3);
  mask.word = (lane < 16 && idx * 32 < d) ? __ldg(words + idx) : 0u;
}

// walk_tiles with the tile's indicator bytes travelling along: body(tile_values, mask, k).
// Without a mask (kMasked false) no byte is loaded and every nibble reads as selected.
template <bool kMasked, class Body>
__device__ __forceinline__ void walk_tiles_masked(const float* __restrict__ row, const uint32_t* __restrict__ ind8,
                                                  uint64_t d, uint32_t k0, uint32_t k1, int j, Body&& body) {
  float4 a[kTileRows], b[kTileRows];
  TileMask ma, mb;
  ma.word = mb.word = 0xffffffffu;
  load_tile(row, static_cast<uint64_t>(k0) * kTile, d, j, a);
  if (kMasked) load_tile_mask(ind8, d, k0, j, ma);
  uint32_t k = k0;
  while (true) {
    if (k + 1 < k1) {
      load_tile(row, static_cast<uint64_t>(k + 1) * kTile, d, j, b);
      if (kMasked) load_tile_mask(ind8, d, k + 1, j, mb);
    }
    body(a, ma, k);
    if (++k >= k1) break;
    if (k + 1 < k1) {
      load_tile(row, static_cast<uint64_t>(k + 1) * kTile, d, j, a);
      if (kMasked) load_tile_mask(ind8, d, k + 1, j, ma);
    }
    body(b, mb, k);
    if (++k >= k1) break;
  }
}

// The CTA's whole share of a launch as one stream of tiles: items blockIdx.x, blockIdx.x + gridDim.x, ...
// (item = worker m, chunk c), each a run of tiles.  The loads of the next tile are issued before the
// current one is processed, across item boundaries too, so the memory pipeline never drains between
// items (at small and medium d an item is only a few tiles long).
//   begin(m, c)            before the first tile of an item
//   body(values, mask, k)  every tile
//   end(m, c, n_tiles)     after the last tile of an item (may synchronise the CTA)
struct ItemPos {
  uint32_t item, m, c, k0, k1;
};
__device__ __forceinline__ ItemPos item_pos(const Geometry& geo, uint32_t item) {
  ItemPos p;
  p.item = item;
  p.m = item / geo.chunks;
  p.c = item - p.m * geo.chunks;
  p.k0 = p.c * geo.group;
  p.k1 = min(p.k0 + geo.group, geo.tiles);
  return p;
}

// kEarlyLoad: the first tile's loads go out before chain_wait() (the gradients are not written by the launch
// this one is chained to); otherwise the caller has waited already.
template <bool kMasked, bool kEarlyLoad = false, class Begin, class Body, class End>
__device__ __forceinline__ void stream_items(const float* __restrict__ g, const uint32_t* __restrict__ indicators,
                                             const Geometry& geo, int j, Begin&& begin, Body&& body, End&& end) {
  const uint32_t n_items = geo.M * geo.chunks;
  if (blockIdx.x >= n_items) {
    if (kEarlyLoad) {
      chain_wait();
      chain_trigger();
    }
    return;
  }
  const uint64_t ind_words = (geo.d + 31) >> 5;
  ItemPos cur = item_pos(geo, blockIdx.x);
  uint32_t k = cur.k0;
  float4 a[kTileRows], b[kTileRows];
  TileMask ma, mb;
  ma.word = mb.word = 0xffffffffu;
  auto load = [&](const ItemPos& p, uint32_t kk, float4 (&v)[kTileRows], TileMask& mk) {
    load_tile(g + static_cast<uint64_t>(p.m) * geo.ld, static_cast<uint64_t>(kk) * kTile, geo.d, j, v);
    if (kMasked)
      load_tile_mask(indicators + static_cast<uint64_t>(p.m) * ind_words, geo.d, kk, j, mk);
  };
  load(cur, k, a, ma);
  if (kEarlyLoad) {
    chain_wait();
    chain_trigger();
  }
  begin(cur.m, cur.c);
  auto step = [&](float4 (&cv)[kTileRows], TileMask& cm, float4 (&nv)[kTileRows], TileMask& nm) -> bool {
    ItemPos nxt = cur;
    uint32_t nk = k + 1;
    bool has_next = true;
    if (nk >= cur.k1) {
      const uint32_t ni = cur.item + gridDim.x;
      has_next = ni < n_items;
      if (has_next) {
        nxt = item_pos(geo, ni);
        nk = nxt.k0;
      }
    }
    if (has_next) load(nxt, nk, nv, nm);
    body(cv, cm, k);
    if (k + 1 >= cur.k1) {
      end(cur.m, cur.c, cur.k1 - cur.k0);
      if (has_next) begin(nxt.m, nxt.c);
    }
    cur = nxt;
    k = nk;
    return has_next;
  };
  while (step(a, ma, b, mb) && step(b, mb, a, ma)) {
  }
}

// ------------------------------------------------------------------ pass B helpers
// Code byte of four coordinates, built on the FMA pipe.  pos/neg are 1.0f or 0.0f per
// coordinate (code 1 = +1, code 2 = -1); the byte value pos0 + 2 neg0 + 4 pos1 + ... + 128 neg3
// is accumulated on top of 2^23, where an fp32's low mantissa bits are the integer itself.
struct CodeBits {
  float pos, neg;
};
__device__ __forceinline__ CodeBits split_code(float v, bool keep) {
  CodeBits c;
  c.pos = (keep && v > 0.f) ? 1.f : 0.f;
  c.neg = (keep && v < 0.f) ? 1.f : 0.f;
  return c;
}
__device__ __forceinline__ uint32_t pack4(CodeBits c0, CodeBits c1, CodeBits c2, CodeBits c3) {
  float b = 8388608.f;
  b = fmaf(c0.pos, 1.f, b);
  b = fmaf(c0.neg, 2.f, b);
  b = fmaf(c1.pos, 4.f, b);
  b = fmaf(c1.neg, 8.f, b);
  b = fmaf(c2.pos, 16.f, b);
  b = fmaf(c2.neg, 32.f, b);
  b = fmaf(c3.pos, 64.f, b);
  b = fmaf(c3.neg, 128.f, b);
  return __float_as_uint(b) & 0xffu;
}

// Number of non-zero 2-bit codes in a byte.
__device__ __forceinline__ uint32_t nonzero_codes(uint32_t byte) {
  return __popc((byte | (byte >> 1)) & 0x55u);
}

// Writes the code bytes of the thread's four rows of tile k.  codes8 is the worker's code
// row; only the last tile can reach past the row's last byte.  The stores are streaming
// (evict-first): the codes are read back only after the whole gradient has gone by.
__device__ __forceinline__ void store_code_bytes(uint8_t* __restrict__ codes8, uint32_t k, int j,
                                                 bool full, uint64_t row_bytes,
                                                 const uint32_t (&bytes)[kTileRows]) {
  const uint64_t b0 = static_cast<uint64_t>(k) * (kTile / 4) + j;
  if (full) {
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) __stcs(codes8 + b0 + r * (kTileCols / 4), static_cast<uint8_t>(bytes[r]));
  } else {
#pragma unroll
    for (int r = 0; r < kTileRows; ++r)
      if (b0 + r * (kTileCols / 4) < row_bytes) __stcs(codes8 + b0 + r * (kTileCols / 4), static_cast<uint8_t>(bytes[r]));
  }
}

// Sums per-thread counts over the CTA; the result is valid in thread 0.
__device__ __forceinline__ unsigned long long block_count(uint32_t cnt, uint32_t* sm_cnt) {
  cnt = __reduce_add_sync(0xffffffffu, cnt);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) sm_cnt[threadIdx.x >> 5] = cnt;
  __syncthreads();
  unsigned long long total = 0;
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) total += sm_cnt[w];
  }
  return total;
}

// Last-CTA epilogue shared by both code kernels: per-worker totals of the counts, and for
// the threshold quantizer the scale s_m = P_m / n_m.
// sm_scales: if given, the CTA's shared copy of the M scales (valid after the CTA's next barrier).
template <bool kThreshold, int kRounds = 4>
__device__ __forceinline__ void finish_codes(const Geometry& geo, const Workspace& ws,
                                             float* scales_out, unsigned long long* counts_out,
                                             float* sm_scales = nullptr) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t m = warp; m < geo.M; m += kThreads / 32) {
    unsigned long long n = 0;
    for (uint32_t idx = lane; idx < geo.chunks; idx += 32)
      n += __ldcg(ws.part_cnt + static_cast<uint64_t>(m) * kMaxChunks + idx);
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) n += __shfl_xor_sync(0xffffffffu, n, s);
    float scale;
    if (kThreshold) {
      const double picked =
          warp_chunk_tree<kRounds>(ws.part_sum + static_cast<uint64_t>(m) * kMaxChunks, geo.chunks, lane);
      scale = n ? static_cast<float>(picked / static_cast<double>(n)) : 0.f;
    } else {
      scale = ws.scales[m];
    }
    if (lane == 0) {
      ws.counts[m] = n;
      if (kThreshold) ws.scales[m] = scale;
      if (scales_out) scales_out[m] = scale;
      if (counts_out) counts_out[m] = n;
      if (sm_scales) sm_scales[m] = scale;
    }
  }
}

// ------------------------------------------------------------------ Philox4x32-10
// Salmon, Moraes, Dror, Shaw, "Parallel random numbers: as easy as 1, 2, 3" (SC'11):
// ten rounds of  (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)),
// the key advancing by the Weyl constants between rounds.
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, uint32_t k0, uint32_t k1) {
  constexpr uint32_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u;
  constexpr uint32_t kW0 = 0x9E3779B9u, kW1 = 0xBB67AE85u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint32_t hi0 = __umulhi(kM0, c.x), lo0 = kM0 * c.x;
    const uint32_t hi1 = __umulhi(kM1, c.z), lo1 = kM1 * c.z;
    c = make_uint4(hi1 ^ c.y ^ k0, lo1, hi0 ^ c.w ^ k1, lo0);
    k0 += kW0;
    k1 += kW1;
  }
  return c;
}

// The same block function with the key schedule (k0 + r*W0, k1 + r*W1), r = 0..9, worked out once on the host
// and passed by value: the twenty words are then constant operands of the xors, and a round is two widening
// multiplies and two three-input xors.
struct PhiloxKeys {
  uint32_t k0[10], k1[10];
};
inline PhiloxKeys philox_key_schedule(uint64_t seed) {
  PhiloxKeys ks;
  uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    ks.k0[r] = k0;
    ks.k1[r] = k1;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  return ks;
}
__device__ __forceinline__ uint4 philox4x32_10(uint4 c, const PhiloxKeys& ks) {
  constexpr uint64_t kM0 = 0xD2511F53u, kM1 = 0xCD9E8D57u;
#pragma unroll
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = kM0 * c.x, p1 = kM1 * c.z;
    c = make_uint4(static_cast<uint32_t>(p1 >> 32) ^ c.y ^ ks.k0[round], static_cast<uint32_t>(p1),
                   static_cast<uint32_t>(p0 >> 32) ^ c.w ^ ks.k1[round], static_cast<uint32_t>(p0));
  }
  return c;
}

// The stochastic quantizer keeps a coordinate iff u < RN(a / s) (fp32 division), a = |v|, u = k 2^-24 with
// k = word >> 8.  The division is avoided where its outcome is certain.  With r24 = RN(1/s) 2^24 and
// q = RN(a r24), q is within 2^-22 q (at most 4 for q <= 2^24; + 2^-124 where the quotient is subnormal) of
// RN(a / s) 2^24, and u < p is k < ceil(p 2^24) for the integer k; so with K = ceil(q), wherever k is more than
// 9 away from K, k < K decides.  A row of four coordinates takes the divisions only if one of its four is
// within 9 (about one row in 200,000).  `fast` is false where 1/s would not be a normal number accurate to
// 2^-24 (s = 0, huge, tiny or not finite): then every row takes the divisions.  A NaN magnitude gives K = 0:
// not kept on either path.
struct KeepTest {
  float s, r24;
  bool fast;
};
__device__ __forceinline__ KeepTest keep_test(float s) {
  KeepTest kt;
  kt.s = s;
  kt.fast = s >= 7.8886090522101181e-31f && s <= 1.2676506002282294e30f;  // 2^-100 <= s <= 2^100
  kt.r24 = kt.fast ? __frcp_rn(s) * 16777216.f : 0.f;
  return kt;
}
// hi32(a * b) + c as one multiply-add (the multiply pipe, not the integer pipe that the Philox xors keep busy).
__device__ __forceinline__ uint32_t mad_hi(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t r;
  asm("mad.hi.u32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(c));
  return r;
}
// k - K for one coordinate (k = word >> 8 = hi32(word * 2^24)): negative iff the fast test keeps it;
// `nearest` collects min |k - K| + 9 as unsigned.
__device__ __forceinline__ uint32_t keep_margin(uint32_t word, float a, const KeepTest& kt, uint32_t& nearest) {
  const uint32_t K = static_cast<uint32_t>(__float2int_ru(__fmul_rn(a, kt.r24)));  // a >= 0: K >= 0
  const uint32_t t = mad_hi(word, 1u << 24, 0u - K);
  nearest = min(nearest, t + 9u);
  return t;
}
__device__ __forceinline__ bool keeps_exact(uint32_t word, float a, float s) {
  return static_cast<float>(word >> 8) * 5.9604644775390625e-08f < __fdiv_rn(a, s);
}
// 2-bit code (1 = +1, 2 = -1, 0 = dropped) from the keep bit (1 or 0) and the sign bit of v; a kept
// coordinate is never +-0.
__device__ __forceinline__ uint32_t code_of(float v, uint32_t keep01) {
  return keep01 * mad_hi(__float_as_uint(v), 2u, 0u) + keep01;
}
// The code byte of four coordinates that share the Philox block w.
__device__ __forceinline__ uint32_t stochastic_code_byte(const float4& v, const uint4& w, const KeepTest& kt) {
  uint32_t nearest = 0xffffffffu;
  const uint32_t tx = keep_margin(w.x, fabsf(v.x), kt, nearest), ty = keep_margin(w.y, fabsf(v.y), kt, nearest);
  const uint32_t tz = keep_margin(w.z, fabsf(v.z), kt, nearest), tw = keep_margin(w.w, fabsf(v.w), kt, nearest);
  uint32_t kx = mad_hi(tx, 2u, 0u), ky = mad_hi(ty, 2u, 0u);  // the sign bit of k - K
  uint32_t kz = mad_hi(tz, 2u, 0u), kw = mad_hi(tw, 2u, 0u);
  if (!kt.fast || nearest <= 18u) {
    kx = keeps_exact(w.x, fabsf(v.x), kt.s) ? 1u : 0u;
    ky = keeps_exact(w.y, fabsf(v.y), kt.s) ? 1u : 0u;
    kz = keeps_exact(w.z, fabsf(v.z), kt.s) ? 1u : 0u;
    kw = keeps_exact(w.w, fabsf(v.w), kt.s) ? 1u : 0u;
  }
  return code_of(v.x, kx) + 4u * code_of(v.y, ky) + 16u * code_of(v.z, kz) + 64u * code_of(v.w, kw);
}

__device__ __forceinline__ float philox_uniform(uint32_t word) {
  return static_cast<float>(word >> 8) * 5.9604644775390625e-08f;  // 2^-24, exact
}

}  // namespace qasg

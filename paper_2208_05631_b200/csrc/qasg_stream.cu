// Passes A and B of the quantizer as ONE launch, for rows that fit the L2 cache.
//
// The threshold Delta_m (Section 3.5) needs the sum over worker m's whole gradient before any of
// its codes can be cut, so a gradient is read twice.  With two kernels (all rows summed, then all rows
// coded) the second read comes from HBM again whenever the M rows together are larger than L2.  Here one
// persistent grid walks the work in the order
//     A(0) .. A(L-1) | A(L) B(0) | A(L+1) B(1) | ... | B(M-L) .. B(M-1)        (A = sum, B = codes)
// so a row is coded while it is still in L2, L rows after it was summed: the M gradients of a
// coordinate cross HBM once.  Items (a worker's chunk of tiles, summed or coded) are dealt to the CTAs
// round-robin in that order; the CTA that completes a worker's last sum item combines the partials and
// publishes Delta_m, and a code item of that worker waits for it.
//
// Forward progress: the launch is cooperative (all CTAs resident), every CTA takes its items in the
// global order, sum items never wait, and a code item waits only for sum items that come earlier in
// that order, so the earliest unfinished item can always run.  Every wait is bounded all the same: after
// max_polls polls the CTA raises kFlagTimeout and the call's abort word, and every CTA returns at its
// next wait (codes of that call are then incomplete and the host learns it from the status word).
//
// The sums are the fixed-order sums of the two-kernel path (same tiles, same trees, same partial
// slots): the results are bit-identical.
#include "qasg_device.cuh"

namespace qasg {

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
__device__ __noinline__ bool wait_for_value(const unsigned int* flag, unsigned int value, unsigned int* abort_word,
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

struct StreamItem {
  uint32_t index, kind, m, c, k0, k1;  // kind 0 = sum (A), 1 = codes (B)
};

__device__ __forceinline__ StreamItem stream_item(const Geometry& geo, uint32_t lag, uint32_t i) {
  const uint32_t ch = geo.chunks;
  StreamItem it;
  it.index = i;
  const uint32_t head = lag * ch;  // stages 0 .. lag-1 hold sum items only
  if (i < head) {
    it.kind = 0;
    it.m = i / ch;
    it.c = i - it.m * ch;
  } else {
    uint32_t r = i - head;
    const uint32_t mid = (geo.M - lag) * 2u * ch;  // stages lag .. M-1: A(s), then B(s - lag)
    if (r < mid) {
      const uint32_t s = r / (2u * ch), q = r - s * 2u * ch;
      it.kind = q < ch ? 0u : 1u;
      it.m = q < ch ? lag + s : s;
      it.c = q < ch ? q : q - ch;
    } else {  // stages M .. M+lag-1: code items only
      r -= mid;
      const uint32_t s = r / ch;
      it.kind = 1;
      it.m = geo.M - lag + s;
      it.c = r - s * ch;
    }
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

// kStochastic: A takes max|g| (the scaler), B draws Philox codes; else A sums |g| (Delta), B cuts Q_Delta.
// kKeepCodes: the code bytes are written with ordinary stores (kept in L2), else with streaming stores.
template <bool kStochastic, bool kKeepCodes>
__global__ void __launch_bounds__(kThreads, 4)
quantize_stream_kernel(const float* __restrict__ g, Geometry geo, StreamParams sp, Workspace ws, StreamSync* sync,
                       uint32_t* __restrict__ codes, float* __restrict__ scales_out,
                       float* __restrict__ thresholds_out, unsigned long long* __restrict__ counts_out) {
  __shared__ ChunkSumStorage sm_sum;
  __shared__ uint32_t sm_cnt[kThreads / 32];
  __shared__ bool sm_flag;
  const int j = threadIdx.x, warp = j >> 5, lane = j & 31;
  const uint32_t total = 2u * geo.M * geo.chunks;
  if (blockIdx.x >= total) return;
  const uint64_t row_words = (geo.d + 15) >> 4;
  const uint32_t full_tiles = static_cast<uint32_t>(geo.d / kTile);
  const uint32_t key0 = static_cast<uint32_t>(sp.seed), key1 = static_cast<uint32_t>(sp.seed >> 32);
  const uint32_t t_lo = static_cast<uint32_t>(sp.t), t_hi = static_cast<uint32_t>(sp.t >> 32);
  ChunkSum chunk_sum(&sm_sum);

  // state of the item being processed
  uint8_t* codes8 = nullptr;
  float level = 0.f, nlevel = 0.f, cntf = 0.f;  // B: Delta_m and -Delta_m (threshold) or s_m (stochastic); kept count
  uint32_t best = 0u, cnt = 0u;                 // stochastic: A's running maximum, B's kept count

  auto begin = [&](const StreamItem& it) -> bool {
    best = 0u, cnt = 0u, cntf = 0.f;
    if (it.kind == 0) return true;
    if (j == 0) sm_flag = wait_for_value(&sync->ready[it.m], 1u, &sync->abort, ws.status, sp.max_polls);
    __syncthreads();
    if (!sm_flag) return false;
    codes8 = reinterpret_cast<uint8_t*>(codes + static_cast<uint64_t>(it.m) * row_words);
    level = kStochastic ? __ldcg(ws.scales + it.m) : __ldcg(ws.thresholds + it.m);
    nlevel = -level;
    return true;
  };

  auto body_a = [&](const float4 (&v)[kTileRows]) {
    if (kStochastic) {
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        best = max(best, __float_as_uint(fabsf(v[r].x)));
        best = max(best, __float_as_uint(fabsf(v[r].y)));
        best = max(best, __float_as_uint(fabsf(v[r].z)));
        best = max(best, __float_as_uint(fabsf(v[r].w)));
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
      chunk_sum.add_tile((cx + cy) + (cz + cw));
    }
  };

  auto body_b = [&](const float4 (&v)[kTileRows], uint32_t m, uint32_t k) {
    uint32_t bytes[kTileRows];
    if (kStochastic) {
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        const float4 t = v[r];
        const uint32_t blk = k * (kTile / 4) + r * (kTileCols / 4) + j;
        const uint4 w = philox4x32_10(make_uint4(blk, sp.stream_base + m, t_lo, t_hi), key0, key1);
        const bool kx = philox_uniform(w.x) < __fdiv_rn(fabsf(t.x), level);
        const bool ky = philox_uniform(w.y) < __fdiv_rn(fabsf(t.y), level);
        const bool kz = philox_uniform(w.z) < __fdiv_rn(fabsf(t.z), level);
        const bool kw = philox_uniform(w.w) < __fdiv_rn(fabsf(t.w), level);
        bytes[r] = pack4(split_code(t.x, kx), split_code(t.y, ky), split_code(t.z, kz), split_code(t.w, kw));
        cnt += nonzero_codes(bytes[r]);
      }
    } else {
      double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
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
      chunk_sum.add_tile((cx + cy) + (cz + cw));
    }
    if (kKeepCodes)
      store_code_bytes_cached(codes8, k, j, k < full_tiles, row_words * 4, bytes);
    else
      store_code_bytes(codes8, k, j, k < full_tiles, row_words * 4, bytes);
  };

  // Takes the worker's ticket after this CTA's partial has been written; true in every thread of the
  // CTA that completed the worker's last item of this kind.
  auto last_of_worker = [&](unsigned int* ticket) -> bool {
    if (j == 0) {
      __threadfence();
      sm_flag = atomicAdd(ticket, 1u) == geo.chunks - 1;
    }
    __syncthreads();
    const bool last = sm_flag;
    if (last) __threadfence();
    return last;
  };

  auto end_a = [&](const StreamItem& it) {
    const uint64_t slot = static_cast<uint64_t>(it.m) * kMaxChunks + it.c;
    if (kStochastic) {
      best = __reduce_max_sync(0xffffffffu, best);
      __syncthreads();
      if (lane == 0) sm_cnt[warp] = best;
      __syncthreads();
      if (j == 0) {
        uint32_t bmax = sm_cnt[0];
#pragma unroll
        for (int w = 1; w < kThreads / 32; ++w) bmax = max(bmax, sm_cnt[w]);
        ws.part_max[slot] = bmax;
      }
    } else {
      const double total_sum = chunk_sum.finish(geo.log2_group);
      if (j == 0) ws.part_sum[slot] = total_sum;
    }
    if (!last_of_worker(&sync->ticket_a[it.m])) return;
    if (warp == 0) {  // one warp combines the worker's chunk partials and publishes the statistic
      if (kStochastic) {
        uint32_t bmax = 0u;
        for (uint32_t idx = lane; idx < geo.chunks; idx += 32)
          bmax = max(bmax, __ldcg(ws.part_max + static_cast<uint64_t>(it.m) * kMaxChunks + idx));
        bmax = __reduce_max_sync(0xffffffffu, bmax);
        if (lane == 0) {
          ws.scales[it.m] = __uint_as_float(bmax);
          ws.thresholds[it.m] = 0.f;
          if (thresholds_out) thresholds_out[it.m] = 0.f;
          if (bmax >= 0x7f800000u) atomicOr(ws.status, kFlagNonFinite);
        }
      } else {
        const double s = warp_chunk_tree(ws.part_sum + static_cast<uint64_t>(it.m) * kMaxChunks, geo.chunks, lane);
        if (lane == 0) {
          const float delta = static_cast<float>((static_cast<double>(sp.coef) * s) / static_cast<double>(geo.d));
          ws.thresholds[it.m] = delta;
          if (thresholds_out) thresholds_out[it.m] = delta;
          if (!isfinite(s)) atomicOr(ws.status, kFlagNonFinite);
        }
      }
      if (lane == 0) {
        sync->ticket_a[it.m] = 0u;  // as the next call expects it
        __threadfence();
        store_release(&sync->ready[it.m], 1u);
      }
    }
  };

  auto end_b = [&](const StreamItem& it) {
    const uint64_t slot = static_cast<uint64_t>(it.m) * kMaxChunks + it.c;
    double picked = 0.0;
    if (!kStochastic) picked = chunk_sum.finish(geo.log2_group);
    const unsigned long long n_item = block_count(kStochastic ? cnt : static_cast<uint32_t>(cntf), sm_cnt);
    if (j == 0) {
      if (!kStochastic) ws.part_sum[slot] = picked;
      ws.part_cnt[slot] = n_item;
    }
    if (!last_of_worker(&sync->ticket_b[it.m])) return;
    if (warp == 0) {  // the worker's count, and for Q_Delta its scale s_m = P_m / n_m
      unsigned long long n = 0;
      for (uint32_t idx = lane; idx < geo.chunks; idx += 32)
        n += __ldcg(ws.part_cnt + static_cast<uint64_t>(it.m) * kMaxChunks + idx);
#pragma unroll
      for (int s = 16; s > 0; s >>= 1) n += __shfl_xor_sync(0xffffffffu, n, s);
      float scale;
      if (kStochastic) {
        scale = level;
      } else {
        const double p = warp_chunk_tree(ws.part_sum + static_cast<uint64_t>(it.m) * kMaxChunks, geo.chunks, lane);
        scale = n ? static_cast<float>(p / static_cast<double>(n)) : 0.f;
      }
      if (lane == 0) {
        ws.counts[it.m] = n;
        if (!kStochastic) ws.scales[it.m] = scale;
        if (scales_out) scales_out[it.m] = scale;
        if (counts_out) counts_out[it.m] = n;
        // every code item of the worker has passed its wait: both words go back to what the next call
        // (or the next replay of a captured launch) expects
        sync->ticket_b[it.m] = 0u;
        sync->ready[it.m] = 0u;
      }
    }
  };

  StreamItem cur = stream_item(geo, sp.lag, blockIdx.x);
  uint32_t k = cur.k0;
  float4 a[kTileRows], b[kTileRows];
  load_tile(g + static_cast<uint64_t>(cur.m) * geo.ld, static_cast<uint64_t>(k) * kTile, geo.d, j, a);
  if (!begin(cur)) return;
  auto step = [&](float4 (&cv)[kTileRows], float4 (&nv)[kTileRows]) -> bool {
    StreamItem nxt = cur;
    uint32_t nk = k + 1;
    bool has_next = true;
    if (nk >= cur.k1) {
      const uint32_t ni = cur.index + gridDim.x;
      has_next = ni < total;
      if (has_next) {
        nxt = stream_item(geo, sp.lag, ni);
        nk = nxt.k0;
      }
    }
    // the next tile's loads go out before this tile is processed, and before any wait: g is an input
    if (has_next) load_tile(g + static_cast<uint64_t>(nxt.m) * geo.ld, static_cast<uint64_t>(nk) * kTile, geo.d, j, nv);
    if (cur.kind == 0)
      body_a(cv);
    else
      body_b(cv, cur.m, k);
    if (k + 1 >= cur.k1) {
      if (cur.kind == 0)
        end_a(cur);
      else
        end_b(cur);
      if (has_next && !begin(nxt)) return false;
    }
    cur = nxt;
    k = nk;
    return has_next;
  };
  while (step(a, b) && step(b, a)) {
  }
}

// A wait that nothing ends: the bounded wait above on a word that no one sets.  The kernel returns after
// max_polls polls with kFlagTimeout raised; nothing else is touched.
__global__ void wait_selftest_kernel(StreamSync* sync, unsigned int* status, uint32_t max_polls) {
  if (threadIdx.x == 0) {
    sync->probe_abort = 0u;
    wait_for_value(&sync->probe, 0xFFFFFFFFu, &sync->probe_abort, status, max_polls);
  }
}

namespace {
template <bool kStochastic, bool kKeepCodes>
cudaError_t launch_stream_as(const float* g, const Geometry& geo, const StreamParams& sp, const Workspace& ws,
                             StreamSync* sync, uint32_t* codes, float* scales_out, float* thresholds_out,
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
  const uint64_t total = 2ull * geo.M * geo.chunks;
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
  return cudaLaunchKernelEx(&cfg, kernel, g, geo, sp, ws, sync, codes, scales_out, thresholds_out, counts_out);
}
}  // namespace

int launch_quantize_stream(bool stochastic, bool keep_codes, const float* g, const Geometry& geo,
                           const StreamParams& sp, const Workspace& ws, StreamSync* sync, uint32_t* codes,
                           float* scales_out, float* thresholds_out, unsigned long long* counts_out,
                           const LaunchShape& shape, cudaStream_t stream) {
  if (stochastic) {
    if (keep_codes)
      launch_stream_as<true, true>(g, geo, sp, ws, sync, codes, scales_out, thresholds_out, counts_out, shape, stream);
    else
      launch_stream_as<true, false>(g, geo, sp, ws, sync, codes, scales_out, thresholds_out, counts_out, shape, stream);
  } else {
    if (keep_codes)
      launch_stream_as<false, true>(g, geo, sp, ws, sync, codes, scales_out, thresholds_out, counts_out, shape, stream);
    else
      launch_stream_as<false, false>(g, geo, sp, ws, sync, codes, scales_out, thresholds_out, counts_out, shape, stream);
  }
  return 1;
}

int launch_wait_selftest(StreamSync* sync, unsigned int* status, uint32_t max_polls, cudaStream_t stream) {
  wait_selftest_kernel<<<1, 32, 0, stream>>>(sync, status, max_polls);
  return 1;
}

}  // namespace qasg

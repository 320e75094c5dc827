// Kernels of the quantized adaptive-subgradient step for sm_100a.
//
//   pass A  abs_sum_kernel / abs_max_kernel     per-worker sum|g| -> Delta_m, or max|g| -> s_m
//   pass B  threshold_codes_kernel              ternary codes, packed; s_m = mean of kept |g|
//           stochastic_codes_kernel             unbiased ternary codes from Philox draws
//   pass C  decode_update_kernel                decode + average + accumulator + QCMD/QRDA (or the
//                                               average alone), dense_update_kernel: update from a dense q
//           decode_update_wide_kernel           the same with eight coordinates per thread (13 to 32 workers, some fewer)
//   server  avg_abs_sum/avg_abs_max/avg_codes   double quantization: Q applied to the average
//   select  select_stats, indicator_or          sparse selection: indicators, statistics over the selected
//
// All three passes are HBM streams.  Passes A and B walk each worker's gradient in
// 4096-coordinate tiles with 128-bit loads (thread j owns columns 4j..4j+3 of each of
// the tile's 4 rows) and keep one tile of loads in flight ahead of the arithmetic.  The
// sums that decide Delta_m and s_m are taken in a fixed order that does not depend on
// the grid: column sums down the rows, a pairwise tree over the 1024 columns (in-thread,
// warp butterfly, across warps), a pairwise tree over tiles.  The CTA that finishes last
// combines the per-chunk partials, so no extra launch or host round trip is needed.
#include "qasg_device.cuh"

namespace qasg {

// ------------------------------------------------------------------ geometry
Geometry make_geometry(uint64_t d, uint64_t ld, uint32_t M, uint32_t max_chunks, uint32_t target_items) {
  Geometry geo;
  geo.d = d;
  geo.ld = ld;
  geo.M = M;
  geo.tiles = static_cast<uint32_t>((d + kTile - 1) / kTile);
  uint32_t group = 1, lg = 0;
  while ((geo.tiles + group - 1) / group > max_chunks) {
    group <<= 1;
    ++lg;
  }
  // Longer chunks while there are still at least target_items of them in the launch: an item pays a
  // CTA-wide combine and a partial write, which a single tile does not amortise.  Any aligned
  // power-of-two grouping is a subtree of the same pairwise tree, so the sums do not change.
  while (target_items && static_cast<uint64_t>(M) * ((geo.tiles + 2 * group - 1) / (2 * group)) >= target_items) {
    group <<= 1;
    ++lg;
  }
  geo.group = group;
  geo.log2_group = lg;
  geo.chunks = (geo.tiles + group - 1) / group;
  return geo;
}

// ------------------------------------------------------------------ pass A: sum |g|
// The CTA's share of the (worker, chunk) items: each chunk's fixed-order sum into its partial slot.
__device__ __forceinline__ void abs_sum_partials(const float* __restrict__ g, const Geometry& geo, const Workspace& ws,
                                                 ChunkSumStorage* sm_sum) {
  const int j = threadIdx.x;
  ChunkSum chunk_sum(sm_sum);
  auto begin = [](uint32_t, uint32_t) {};
  auto body = [&](const float4 (&v)[kTileRows], const TileMask&, uint32_t) {
        double cx = fabsf(v[0].x), cy = fabsf(v[0].y), cz = fabsf(v[0].z), cw = fabsf(v[0].w);
#pragma unroll
        for (int r = 1; r < kTileRows; ++r) {
          cx += static_cast<double>(fabsf(v[r].x));
          cy += static_cast<double>(fabsf(v[r].y));
          cz += static_cast<double>(fabsf(v[r].z));
          cw += static_cast<double>(fabsf(v[r].w));
        }
        chunk_sum.add_tile((cx + cy) + (cz + cw));
      };
  auto end = [&](uint32_t m, uint32_t c, uint32_t) {
        const double total = chunk_sum.finish(geo.log2_group);
        if (j == 0) ws.part_sum[static_cast<uint64_t>(m) * kMaxChunks + c] = total;
      };
  stream_items<false>(g, nullptr, geo, j, begin, body, end);
}

// Delta_m of every worker from the chunk partials (all of them written and visible): one warp per worker.
template <int kRounds = 4>
__device__ __forceinline__ void abs_sum_combine(const Geometry& geo, float coef, const Workspace& ws,
                                                float* __restrict__ thresholds_out,
                                                const unsigned long long* __restrict__ denom) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t m = warp; m < geo.M; m += kThreads / 32) {
    const double total =
        warp_chunk_tree<kRounds>(ws.part_sum + static_cast<uint64_t>(m) * kMaxChunks, geo.chunks, lane);
    if (lane == 0) {
      // the mean is over all d coordinates, or over the selected ones when a count is given
      const unsigned long long n = denom ? denom[m] : geo.d;
      const float delta = n ? static_cast<float>((static_cast<double>(coef) * total) / static_cast<double>(n)) : 0.f;
      ws.thresholds[m] = delta;
      if (thresholds_out) thresholds_out[m] = delta;
      if (!isfinite(total)) atomicOr(ws.status, kFlagNonFinite);
    }
  }
}

__global__ void __launch_bounds__(kThreads, 4)
abs_sum_kernel(const float* __restrict__ g, Geometry geo, float coef, Workspace ws,
               float* __restrict__ thresholds_out, const unsigned long long* __restrict__ denom) {
  __shared__ ChunkSumStorage sm_sum;
  __shared__ bool sm_last;
  chain_wait();  // the gradients may come from the launch before this one
  chain_trigger();
  abs_sum_partials(g, geo, ws, &sm_sum);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  abs_sum_combine(geo, coef, ws, thresholds_out, denom);
  if (threadIdx.x == 0) *ws.ticket = 0u;
}

// ------------------------------------------------------------------ pass A': max |g|
__device__ __forceinline__ void abs_max_partials(const float* __restrict__ g, const Geometry& geo, const Workspace& ws,
                                                 uint32_t* sm_warp) {
  const int j = threadIdx.x;
  const uint32_t n_items = geo.M * geo.chunks;
  for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const uint32_t m = item / geo.chunks, c = item - m * geo.chunks;
    const float* row = g + static_cast<uint64_t>(m) * geo.ld;
    const uint32_t k0 = c * geo.group;
    const uint32_t k1 = min(k0 + geo.group, geo.tiles);
    uint32_t best = 0u;  // bit patterns of non-negative floats order like their values
    auto body = [&](const float4 (&v)[kTileRows], uint32_t) {
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        best = max(best, __float_as_uint(fabsf(v[r].x)));
        best = max(best, __float_as_uint(fabsf(v[r].y)));
        best = max(best, __float_as_uint(fabsf(v[r].z)));
        best = max(best, __float_as_uint(fabsf(v[r].w)));
      }
    };
    walk_tiles(row, geo.d, k0, k1, j, body);
    best = __reduce_max_sync(0xffffffffu, best);
    __syncthreads();  // the previous item's readers are done with sm_warp
    if ((j & 31) == 0) sm_warp[j >> 5] = best;
    __syncthreads();
    if (j == 0) {
      uint32_t bmax = sm_warp[0];
#pragma unroll
      for (int w = 1; w < kThreads / 32; ++w) bmax = max(bmax, sm_warp[w]);
      ws.part_max[static_cast<uint64_t>(m) * kMaxChunks + c] = bmax;
    }
  }
}

// s_m = max |g_m| of every worker from the chunk maxima: one warp per worker.
__device__ __forceinline__ void abs_max_combine(const Geometry& geo, const Workspace& ws) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (uint32_t m = warp; m < geo.M; m += kThreads / 32) {
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
}

__global__ void __launch_bounds__(kThreads)
abs_max_kernel(const float* __restrict__ g, Geometry geo, Workspace ws) {
  __shared__ uint32_t sm_warp[kThreads / 32];
  __shared__ bool sm_last;
  chain_wait();
  chain_trigger();
  abs_max_partials(g, geo, ws, sm_warp);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  abs_max_combine(geo, ws);
  if (threadIdx.x == 0) *ws.ticket = 0u;
}

// ------------------------------------------------------------------ pass B: Q_Delta codes
// kMasked: only coordinates whose indicator bit is set are candidates (sparse selection, Q(S(g, I))).
// The CTA's share of the (worker, chunk) items: code bytes, and each chunk's kept sum and count into its
// partial slots.  kEarlyLoad: the first gradient tile is requested ahead of chain_wait().
template <bool kMasked, bool kEarlyLoad>
__device__ __forceinline__ void threshold_codes_partials(const float* __restrict__ g, const Geometry& geo,
                                                         const Workspace& ws, uint32_t* __restrict__ codes,
                                                         const uint32_t* __restrict__ indicators,
                                                         ChunkSumStorage* sm_sum, uint32_t* sm_cnt) {
  const int j = threadIdx.x;
  const uint64_t row_words = (geo.d + 15) >> 4;
  const uint32_t full_tiles = static_cast<uint32_t>(geo.d / kTile);
  ChunkSum chunk_sum(sm_sum);
  uint8_t* codes8 = nullptr;  // per item: the worker's code row, its threshold, the kept count so far
  float delta = 0.f, ndelta = 0.f, cntf = 0.f;
  auto begin = [&](uint32_t m, uint32_t) {
        codes8 = reinterpret_cast<uint8_t*>(codes + static_cast<uint64_t>(m) * row_words);
        delta = ws.thresholds[m];
        ndelta = -delta;
        cntf = 0.f;
      };
  auto body = [&](const float4 (&v)[kTileRows], const TileMask& mask, uint32_t k) {
        double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
        uint32_t bytes[kTileRows];
        auto rows = [&](auto use_mask) {
#pragma unroll
          for (int r = 0; r < kTileRows; ++r) {
            float4 t = v[r];
            if (decltype(use_mask)::value) {  // a coordinate that is not selected is not sent: it enters as +0.0, which codes 0
              const uint32_t nib = mask.nibble(r, j);
              t.x = (nib & 1u) ? t.x : 0.f, t.y = (nib & 2u) ? t.y : 0.f;
              t.z = (nib & 4u) ? t.z : 0.f, t.w = (nib & 8u) ? t.w : 0.f;
            }
            // strict comparisons; a NaN threshold or value compares false and codes 0
            const float px = t.x > delta ? 1.f : 0.f, nx = t.x < ndelta ? 1.f : 0.f;
            const float py = t.y > delta ? 1.f : 0.f, ny = t.y < ndelta ? 1.f : 0.f;
            const float pz = t.z > delta ? 1.f : 0.f, nz = t.z < ndelta ? 1.f : 0.f;
            const float pw = t.w > delta ? 1.f : 0.f, nw = t.w < ndelta ? 1.f : 0.f;
            const float kx = px + nx, ky = py + ny, kz = pz + nz, kw = pw + nw;  // 1.0f where kept
            // |v| * 1 = |v| and |v| * 0 = +0: the kept magnitudes enter the sum unchanged
            cx += static_cast<double>(fabsf(t.x) * kx);
            cy += static_cast<double>(fabsf(t.y) * ky);
            cz += static_cast<double>(fabsf(t.z) * kz);
            cw += static_cast<double>(fabsf(t.w) * kw);
            cntf += (kx + ky) + (kz + kw);  // exact: far below 2^24 per thread and chunk
            bytes[r] = pack4({px, nx}, {py, ny}, {pz, nz}, {pw, nw});
          }
        };
        // A warp whose 512 coordinates of this tile are all selected (its 16 indicator words are all ones)
        // takes the unmasked arithmetic; the decision is the same in every lane.
        if (kMasked && !__all_sync(0xffffffffu, (j & 31) >= 16 || mask.word == 0xffffffffu))
          rows(std::true_type{});
        else
          rows(std::false_type{});
        store_code_bytes(codes8, k, j, k < full_tiles, row_words * 4, bytes);
        chunk_sum.add_tile((cx + cy) + (cz + cw));
      };
  auto end = [&](uint32_t m, uint32_t c, uint32_t) {
        const double picked = chunk_sum.finish(geo.log2_group);
        const unsigned long long total = block_count(static_cast<uint32_t>(cntf), sm_cnt);
        if (j == 0) {
          const uint64_t p = static_cast<uint64_t>(m) * kMaxChunks + c;
          ws.part_sum[p] = picked;
          ws.part_cnt[p] = total;
        }
      };
  stream_items<kMasked, kEarlyLoad>(g, indicators, geo, j, begin, body, end);
}

template <bool kMasked>
__global__ void __launch_bounds__(kThreads, 4)
threshold_codes_kernel(const float* __restrict__ g, Geometry geo, Workspace ws,
                       uint32_t* __restrict__ codes, float* __restrict__ scales_out,
                       unsigned long long* __restrict__ counts_out, const uint32_t* __restrict__ indicators) {
  __shared__ ChunkSumStorage sm_sum;
  __shared__ uint32_t sm_cnt[kThreads / 32];
  __shared__ bool sm_last;
  if (kMasked) {  // the indicator words come from the launch before this one
    chain_wait();
    chain_trigger();
  }
  // unmasked: the first gradient tile is requested ahead of the wait for the thresholds
  threshold_codes_partials<kMasked, !kMasked>(g, geo, ws, codes, indicators, &sm_sum, sm_cnt);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  finish_codes<true>(geo, ws, scales_out, counts_out);
  if (threadIdx.x == 0) *ws.ticket = 0u;
}

// ------------------------------------------------------------------ pass B': stochastic codes
template <bool kMasked>
__device__ __forceinline__ void stochastic_codes_partials(const float* __restrict__ g, const Geometry& geo,
                                                          const PhiloxKeys& keys, uint64_t t, uint32_t stream_base,
                                                          const Workspace& ws, uint32_t* __restrict__ codes,
                                                          const uint32_t* __restrict__ indicators, uint32_t* sm_cnt) {
  const int j = threadIdx.x;
  const uint32_t n_items = geo.M * geo.chunks;
  const uint64_t row_words = (geo.d + 15) >> 4;
  const uint32_t full_tiles = static_cast<uint32_t>(geo.d / kTile);
  const uint32_t t_lo = static_cast<uint32_t>(t), t_hi = static_cast<uint32_t>(t >> 32);
  for (uint32_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const uint32_t m = item / geo.chunks, c = item - m * geo.chunks;
    const float* row = g + static_cast<uint64_t>(m) * geo.ld;
    uint8_t* codes8 = reinterpret_cast<uint8_t*>(codes + static_cast<uint64_t>(m) * row_words);
    const KeepTest kt = keep_test(ws.scales[m]);
    const uint32_t* ind_row = kMasked ? indicators + static_cast<uint64_t>(m) * ((geo.d + 31) >> 5) : nullptr;
    const uint32_t k0 = c * geo.group;
    const uint32_t k1 = min(k0 + geo.group, geo.tiles);
    uint32_t cnt = 0;
    auto body = [&](const float4 (&tile)[kTileRows], const TileMask& mask, uint32_t k) {
      uint32_t bytes[kTileRows];
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        const float4 v = tile[r];
        // coordinates 4*blk .. 4*blk+3 share one Philox block
        const uint32_t blk = k * (kTile / 4) + r * (kTileCols / 4) + j;
        const uint4 w = philox4x32_10(make_uint4(blk, stream_base + m, t_lo, t_hi), keys);
        // u < |v|/s as the IEEE division decides it; s = 0 gives NaN and the comparison is false.
        bytes[r] = stochastic_code_byte(v, w, kt);
        if (kMasked) {  // unselected coordinates code 0: the nibble's bits spread to the byte's four fields
          const uint32_t nib = mask.nibble(r, j);
          bytes[r] &= ((nib & 1u) | ((nib & 2u) << 1) | ((nib & 4u) << 2) | ((nib & 8u) << 3)) * 3u;
        }
        cnt += nonzero_codes(bytes[r]);
      }
      store_code_bytes(codes8, k, j, k < full_tiles, row_words * 4, bytes);
    };

    walk_tiles_masked<kMasked>(row, ind_row, geo.d, k0, k1, j, body);
    const unsigned long long total = block_count(cnt, sm_cnt);
    if (j == 0) ws.part_cnt[static_cast<uint64_t>(m) * kMaxChunks + c] = total;
  }
}

template <bool kMasked>
__global__ void __launch_bounds__(kThreads, 4)
stochastic_codes_kernel(const float* __restrict__ g, Geometry geo, PhiloxKeys keys, uint64_t t,
                        uint32_t stream_base, Workspace ws, uint32_t* __restrict__ codes, float* __restrict__ scales_out,
                        unsigned long long* __restrict__ counts_out, const uint32_t* __restrict__ indicators) {
  __shared__ uint32_t sm_cnt[kThreads / 32];
  __shared__ bool sm_last;
  chain_wait();
  chain_trigger();
  stochastic_codes_partials<kMasked>(g, geo, keys, t, stream_base, ws, codes, indicators, sm_cnt);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  finish_codes<false>(geo, ws, scales_out, counts_out);
  if (threadIdx.x == 0) *ws.ticket = 0u;
}

// ------------------------------------------------------------------ pass C helpers
// Square root and reciprocal from the special-function unit: at most 2 ulp off (relative
// error below 2.4e-7), two orders of magnitude inside the tolerance on the iterates, for a
// fraction of the instructions of the correctly rounded forms.  Subnormals are kept.
__device__ __forceinline__ float sqrt_sfu(float a) {
  float r;
  asm("sqrt.approx.f32 %0, %1;" : "=f"(r) : "f"(a));
  return r;
}
__device__ __forceinline__ float rcp_sfu(float a) {
  float r;
  asm("rcp.approx.f32 %0, %1;" : "=f"(r) : "f"(a));
  return r;
}

// Eq. H_t and Eq. QCMD for one coordinate.
__device__ __forceinline__ void cmd_update(float q, float& x, float& h, const StepScalars& sc) {
  const float hn = fmaf(q, q, h);
  const float big_h = sc.delta + sqrt_sfu(hn);
  const float rate = sc.eta * rcp_sfu(big_h);
  const float u = fmaf(-rate, q, x);
  const float mag = fabsf(u) - sc.lambda * rate;
  x = mag > 0.f ? copysignf(mag, u) : 0.f;
  h = hn;
}

// Eq. H_t and Eq. QRDA for one coordinate.  sc.t holds t, sc.inv_t its reciprocal.
__device__ __forceinline__ void rda_update(float q, float& x, float& h, float& z, const StepScalars& sc) {
  const float hn = fmaf(q, q, h);
  const float zn = z + q;
  const float big_h = sc.delta + sqrt_sfu(hn);
  const float a = fmaf(fabsf(zn), sc.inv_t, -sc.lambda);
  const float coef = (sc.t * sc.eta) * rcp_sfu(big_h);
  x = a > 0.f ? -copysignf(coef * a, zn) : 0.f;
  h = hn;
  z = zn;
}

// The decode keeps, per group of 4 workers, a table of the 256 possible partial sums
//   lut[G][c0 | c1<<2 | c2<<4 | c3<<6] = sum_k scale[4G+k] * value(c_k)     (value: 1 -> +1, 2 -> -1)
// in shared memory, in fp64: terms of opposite sign cancel across workers, and the update
// divides by H = delta + sqrt(h), which can be as small as |q| itself, so q must carry no
// more than its own fp32 rounding error.
// kLanes = 1: one copy, [G][256].  kLanes = 32: one copy per lane, [G][256][32], so that the
// 32 lookups of a warp never meet in a bank (64 KB per group of workers).
template <int kLanes>
__device__ __forceinline__ void build_decode_lut(double* lut, const float* __restrict__ scales, uint32_t M) {
  const uint32_t groups = (M + 3) >> 2;
  for (uint32_t e = threadIdx.x; e < groups * 256 * kLanes; e += blockDim.x) {
    const uint32_t entry = e / kLanes;
    const uint32_t grp = entry >> 8, idx = entry & 255u;
    double acc = 0.0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t m = grp * 4 + k;
      const uint32_t c = (idx >> (2 * k)) & 3u;
      if (m < M && (c == 1u || c == 2u)) {
        const double sv = static_cast<double>(scales[m]);
        acc += (c == 1u) ? sv : -sv;
      }
    }
    lut[e] = acc;
  }
  __syncthreads();
}

// In a word whose byte k holds worker k's four 2-bit codes (coordinates 0..3), exchanges the
// roles of byte and field: afterwards byte c holds the four workers' codes of coordinate c.
__device__ __forceinline__ uint32_t transpose_2bit_4x4(uint32_t w) {
  uint32_t t = ((w >> 6) ^ w) & 0x00CC00CCu;
  w ^= t ^ (t << 6);
  t = ((w >> 12) ^ w) & 0x0000F0F0u;
  w ^= t ^ (t << 12);
  return w;
}

// Averaged decoded gradient of the four coordinates of group `grp` (Eq. SynQ_t).
// kM4 > 0: the number of worker groups ceil(M/4) is a compile-time constant and the loop
// unrolls; kM4 = 0: any M.
// kFresh: the codes were written earlier in this launch (by other CTAs): they are read from L2, not through
// the read-only path.
template <int kM4, int kLanes, bool kFresh = false>
__device__ __forceinline__ float4 decode_group(const uint8_t* __restrict__ codes8, uint64_t row_bytes,
                                               const double* lut, uint32_t M, double inv_m,
                                               uint64_t grp, uint32_t& bad) {
  auto code_byte = [](const uint8_t* q) -> uint32_t { return kFresh ? __ldcg(q) : __ldg(q); };
  double q0 = 0.0, q1 = 0.0, q2 = 0.0, q3 = 0.0;
  const uint32_t m4 = kM4 > 0 ? static_cast<uint32_t>(kM4) : (M + 3) >> 2;
  if (kLanes > 1) lut += threadIdx.x & (kLanes - 1);  // kLanes copies: lanes l and l + kLanes share one
#pragma unroll
  for (uint32_t G = 0; G < m4; ++G) {
    const uint8_t* p = codes8 + grp + static_cast<uint64_t>(4 * G) * row_bytes;
    const bool whole = (kM4 > 0 && G + 1 < m4);  // only the last group can be short of workers
    uint32_t w = code_byte(p);
    if (whole || 4 * G + 1 < M) w |= code_byte(p + row_bytes) << 8;
    if (whole || 4 * G + 2 < M) w |= code_byte(p + 2 * row_bytes) << 16;
    if (whole || 4 * G + 3 < M) w |= code_byte(p + 3 * row_bytes) << 24;
    bad |= w & (w >> 1) & 0x55555555u;
    w = transpose_2bit_4x4(w);
    const double* l = lut + static_cast<size_t>(G) * 256 * kLanes;
    q0 += l[(w & 255u) * kLanes];
    q1 += l[((w >> 8) & 255u) * kLanes];
    q2 += l[((w >> 16) & 255u) * kLanes];
    q3 += l[(w >> 24) * kLanes];
  }
  return make_float4(static_cast<float>(q0 * inv_m), static_cast<float>(q1 * inv_m),
                     static_cast<float>(q2 * inv_m), static_cast<float>(q3 * inv_m));
}

// ------------------------------------------------------------------ pass C: fused
// State of one group of four coordinates.
// kRule: 0 = QCMD, 1 = QRDA, 2 = no update at all: the averaged gradient is written to x.
template <int kRule>
struct GroupState {
  float4 h, xz;  // xz: x for QCMD (read and written), z for QRDA
  __device__ __forceinline__ void load(const float* __restrict__ x, const float* __restrict__ hh,
                                       const float* __restrict__ z, uint64_t grp) {
    if (kRule == 2) return;
    h = *reinterpret_cast<const float4*>(hh + 4 * grp);
    xz = *reinterpret_cast<const float4*>((kRule == 0 ? x : z) + 4 * grp);
  }
  __device__ __forceinline__ void update_store(float4 q, float* __restrict__ x, float* __restrict__ hh,
                                               float* __restrict__ z, uint64_t grp, const StepScalars& sc) {
    if (kRule == 2) {
      *reinterpret_cast<float4*>(x + 4 * grp) = q;
      return;
    }
    if (kRule == 0) {
      cmd_update(q.x, xz.x, h.x, sc);
      cmd_update(q.y, xz.y, h.y, sc);
      cmd_update(q.z, xz.z, h.z, sc);
      cmd_update(q.w, xz.w, h.w, sc);
      *reinterpret_cast<float4*>(x + 4 * grp) = xz;
    } else {
      float4 xv;
      rda_update(q.x, xv.x, h.x, xz.x, sc);
      rda_update(q.y, xv.y, h.y, xz.y, sc);
      rda_update(q.z, xv.z, h.z, xz.z, sc);
      rda_update(q.w, xv.w, h.w, xz.w, sc);
      *reinterpret_cast<float4*>(z + 4 * grp) = xz;
      *reinterpret_cast<float4*>(x + 4 * grp) = xv;
    }
    *reinterpret_cast<float4*>(hh + 4 * grp) = h;
  }
};

// The last group of a vector whose length is not a multiple of 4: d % 4 coordinates, one by one.
template <int kRule>
__device__ __forceinline__ void update_ragged_group(float4 q, uint64_t grp, uint64_t d, float* __restrict__ x,
                                                    float* __restrict__ h, float* __restrict__ z,
                                                    const StepScalars& sc) {
  const float qs[4] = {q.x, q.y, q.z, q.w};
  for (uint64_t c = 4 * grp; c < d; ++c) {
    if (kRule == 2) {
      x[c] = qs[c - 4 * grp];
      continue;
    }
    float xi = (kRule == 0) ? x[c] : 0.f, hi = h[c];
    if (kRule == 0) {
      cmd_update(qs[c - 4 * grp], xi, hi, sc);
    } else {
      float zi = z[c];
      rda_update(qs[c - 4 * grp], xi, hi, zi, sc);
      z[c] = zi;
    }
    x[c] = xi;
    h[c] = hi;
  }
}

// kThreadsC threads per CTA; a CTA takes kGroups * kThreadsC consecutive groups per round and a
// thread owns kGroups of them, kThreadsC apart, with all their loads in flight before it decodes.
// Up to 12 workers run with 16 copies of the tables (512 threads, two CTAs per SM); up to 52 with 16 or 8
// copies and one CTA of 1024 threads per SM; more workers share one table per CTA.
template <int kRule, int kM4, int kLanes, int kThreadsC, int kGroups>
__global__ void __launch_bounds__(kThreadsC)
decode_update_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ scales, uint64_t d,
                     uint32_t M, double inv_m, float* __restrict__ x, float* __restrict__ h,
                     float* __restrict__ z, StepScalars sc, unsigned int* __restrict__ status) {
  extern __shared__ double sm_lut[];
  chain_wait();  // scales and codes come from the launch before this one
  chain_trigger();
  build_decode_lut<kLanes>(sm_lut, scales, M);
  const uint8_t* codes8 = reinterpret_cast<const uint8_t*>(codes);
  const uint64_t row_bytes = ((d + 15) >> 4) * 4;
  const uint64_t groups = (d + 3) >> 2, full = d >> 2;
  const uint64_t stride = static_cast<uint64_t>(gridDim.x) * (kGroups * kThreadsC);
  uint32_t bad = 0;
  for (uint64_t g0 = static_cast<uint64_t>(blockIdx.x) * (kGroups * kThreadsC) + threadIdx.x; g0 < groups;
       g0 += stride) {
    if (g0 + (kGroups - 1) * kThreadsC < full) {
      GroupState<kRule> s[kGroups];
#pragma unroll
      for (int i = 0; i < kGroups; ++i) s[i].load(x, h, z, g0 + i * kThreadsC);
      float4 q[kGroups];
#pragma unroll
      for (int i = 0; i < kGroups; ++i)
        q[i] = decode_group<kM4, kLanes>(codes8, row_bytes, sm_lut, M, inv_m, g0 + i * kThreadsC, bad);
#pragma unroll
      for (int i = 0; i < kGroups; ++i) s[i].update_store(q[i], x, h, z, g0 + i * kThreadsC, sc);
      continue;
    }
    for (int i = 0; i < kGroups; ++i) {  // the last round, group by group
      const uint64_t grp = g0 + static_cast<uint64_t>(i) * kThreadsC;
      if (grp >= groups) break;
      const float4 q = decode_group<kM4, kLanes>(codes8, row_bytes, sm_lut, M, inv_m, grp, bad);
      if (grp < full) {
        GroupState<kRule> s0;
        s0.load(x, h, z, grp);
        s0.update_store(q, x, h, z, grp, sc);
      } else {
        update_ragged_group<kRule>(q, grp, d, x, h, z, sc);
      }
    }
  }
  if (bad) atomicOr(status, kFlagBadCode);
}

// ------------------------------------------------------------------ the whole step in one launch
// Passes A, B and C of a fused step as the phases of one launch, for sizes where three launches cost more
// than the work: the CTAs (all resident: a cooperative launch, or one CTA) meet twice, after the chunk
// partials of pass A and after those of pass B, and at each meeting all workers' thresholds (scales) are
// worked out from the partials: by every CTA for itself when they are few, by the one that arrives last
// when they are many (as the last CTA of the separate kernels does).  Same arithmetic on the same numbers
// either way.  The phases are the functions the three kernels are made of: every output has the bits of
// the three-launch path.
struct FusedParams {
  float coef;            // threshold coefficient (0.75)
  uint32_t max_polls;    // bound of the waits at the meetings
  uint32_t stream_base;  // Philox counter word 1 = stream_base + worker
  uint64_t t;
};

template <bool kStochastic>
__device__ __forceinline__ void fused_phase_a(const float* __restrict__ g, const Geometry& geo, const Workspace& ws,
                                           ChunkSumStorage* sm_sum, uint32_t* sm_cnt) {
  if (kStochastic)
    abs_max_partials(g, geo, ws, sm_cnt);
  else
    abs_sum_partials(g, geo, ws, sm_sum);
}
// kRounds: 1 where one CTA combines for all (it reads up to 1024 partials per worker: one round trip to L2
// instead of four); 4 where every CTA combines for itself (few partials; the small cases measured faster).
template <bool kStochastic, int kRounds>
__device__ __forceinline__ void fused_combine_a(const Geometry& geo, float coef, const Workspace& ws) {
  if (kStochastic)
    abs_max_combine(geo, ws);
  else
    abs_sum_combine<kRounds>(geo, coef, ws, nullptr, nullptr);
}
template <bool kStochastic>
__device__ __forceinline__ void fused_phase_b(const float* __restrict__ g, const Geometry& geo, const PhiloxKeys& keys,
                                           uint64_t t, uint32_t stream_base, const Workspace& wsb,
                                           uint32_t* __restrict__ codes, ChunkSumStorage* sm_sum, uint32_t* sm_cnt) {
  if (kStochastic)
    stochastic_codes_partials<false>(g, geo, keys, t, stream_base, wsb, codes, nullptr, sm_cnt);
  else
    threshold_codes_partials<false, false>(g, geo, wsb, codes, nullptr, sm_sum, sm_cnt);
}
template <bool kStochastic, int kRounds>
__device__ __forceinline__ void fused_combine_b(const Geometry& geo, const Workspace& wsb, float* scales_out,
                                             float* sm_scales) {
  finish_codes<!kStochastic, kRounds>(geo, wsb, scales_out, nullptr, sm_scales);
}

// Two CTAs per SM: the launch is for problems that do not fill the machine, and the phases keep their
// registers (called instead of inlined, or squeezed into 64 registers, the small cases measured 20 % slower).
template <int kRule, bool kStochastic>
__global__ void __launch_bounds__(kThreads, 2)
fused_step_kernel(const float* __restrict__ g, Geometry geo, FusedParams fp, PhiloxKeys keys, Workspace ws,
                  Workspace wsb, StreamSync* sync, uint32_t* __restrict__ codes, float* __restrict__ scales_out,
                  float* __restrict__ x, float* __restrict__ h, float* __restrict__ z, StepScalars sc) {
  extern __shared__ double sm_lut[];  // [ceil(M/4)][256]
  __shared__ ChunkSumStorage sm_sum;
  __shared__ uint32_t sm_cnt[kThreads / 32];
  __shared__ float sm_scales[kMaxWorkers];
  __shared__ uint32_t sm_word;
  const int j = threadIdx.x;
  chain_wait();  // the gradients may come from the launch before this one
  chain_trigger();
  // pass A: chunk partials, then the thresholds (or scalers) of all workers.  (After a launch that gave up
  // no further launch gets past this meeting until the host has cleared the words: qasg_last_async_status
  // does, when it reports the time-out.)
  const bool everyone = gridDim.x <= kMeetEveryone;  // every CTA combines for itself
  fused_phase_a<kStochastic>(g, geo, ws, &sm_sum, sm_cnt);
  if (!grid_meet<false>(sync, 1u, fp.max_polls, ws.status, &sm_word, [&]() {
        if (everyone)
          fused_combine_a<kStochastic, 4>(geo, fp.coef, ws);
        else
          fused_combine_a<kStochastic, 1>(geo, fp.coef, ws);
      }))
    return;

  // pass B: code bytes and chunk partials, then the scales of all workers.  Its partials go to slots of
  // their own (wsb: the statistics of ws, other partial slots).
  fused_phase_b<kStochastic>(g, geo, keys, fp.t, fp.stream_base, wsb, codes, &sm_sum, sm_cnt);
  // where every CTA combines for itself the scales go straight into its shared copy
  if (!grid_meet<true>(sync, 2u, fp.max_polls, ws.status, &sm_word, [&]() {
        if (everyone)
          fused_combine_b<kStochastic, 4>(geo, wsb, blockIdx.x == 0 ? scales_out : nullptr, sm_scales);
        else
          fused_combine_b<kStochastic, 1>(geo, wsb, scales_out, nullptr);
      }))
    return;
  if (!everyone) {
    if (j < static_cast<int>(geo.M)) sm_scales[j] = __ldcg(ws.scales + j);
    __syncthreads();
  }

  // pass C: the CTA's share of the coordinates
  build_decode_lut<1>(sm_lut, sm_scales, geo.M);
  const uint8_t* codes8 = reinterpret_cast<const uint8_t*>(codes);
  const uint64_t row_bytes = ((geo.d + 15) >> 4) * 4;
  const uint64_t groups = (geo.d + 3) >> 2, full = geo.d >> 2;
  const double inv_m = 1.0 / static_cast<double>(geo.M);
  uint32_t bad = 0;
  for (uint64_t grp = static_cast<uint64_t>(blockIdx.x) * kThreads + j; grp < groups;
       grp += static_cast<uint64_t>(gridDim.x) * kThreads) {
    if (grp < full) {
      GroupState<kRule> s0;
      s0.load(x, h, z, grp);
      const float4 q = decode_group<0, 1, true>(codes8, row_bytes, sm_lut, geo.M, inv_m, grp, bad);
      s0.update_store(q, x, h, z, grp, sc);
    } else {
      const float4 q = decode_group<0, 1, true>(codes8, row_bytes, sm_lut, geo.M, inv_m, grp, bad);
      update_ragged_group<kRule>(q, grp, geo.d, x, h, z, sc);
    }
  }
  if (bad) atomicOr(ws.status, kFlagBadCode);
}

// ------------------------------------------------------------------ pass C, eight coordinates per thread
// Serves 13 to 32 workers, and fewer where it was measured faster (the launcher says which).
// With many workers the byte-per-worker decode above is bound by integer instructions (address
// arithmetic for one byte load per worker and four coordinates, the 2-bit transposition, the
// field extraction), not by HBM.  Here a thread owns eight consecutive coordinates, so one
// 16-bit load per worker brings its codes, and the lookup index is formed differently: the four
// bytes gathered from a group of four workers are masked down to one 2-bit field each, and one
// 32-bit multiplication sums them with the weights (1, 3, 9, 27) into the radix-3 index
//   idx = c0 + 3 c1 + 9 c2 + 27 c3  in 0..80      (code values 0, 1, 2).  The table of a worker group then has 81 entries instead of 256, so 16
// lane copies (no bank conflict for 64-bit lookups) fit for every worker count: 10 KB per group.
// The partial sums are the same doubles, added in the same order, as in decode_update_kernel.
// A code value 3 has no radix-3 digit: the fields are tested before they are used, and a thread that
// meets one clears them first (code 3 decodes to 0).
constexpr int kWideThreads = 512;
constexpr int kLut3Entries = 81;
constexpr int kLut3Lanes = 16;

__device__ __forceinline__ void build_decode_lut3(double* lut, const float* __restrict__ scales, uint32_t M) {
  const uint32_t groups = (M + 3) >> 2;
  for (uint32_t e = threadIdx.x; e < groups * kLut3Entries * kLut3Lanes; e += blockDim.x) {
    const uint32_t entry = e / kLut3Lanes;
    const uint32_t grp = entry / kLut3Entries;
    uint32_t idx = entry - grp * kLut3Entries;
    double acc = 0.0;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t m = grp * 4 + k;
      const uint32_t c = idx % 3u;
      idx /= 3u;
      if (m < M && c != 0u) {
        const double sv = static_cast<double>(scales[m]);
        acc += (c == 1u) ? sv : -sv;
      }
    }
    lut[e] = acc;
  }
  __syncthreads();
}

// Entry idx of the lane's copy of the table at shared-memory address table_lane: 32-bit address
// arithmetic, one multiply-add.
__device__ __forceinline__ double lut3_entry(uint32_t table_lane, uint32_t idx) {
  double v;
  asm("ld.shared.f64 %0, [%1];" : "=d"(v) : "r"(idx * (kLut3Lanes * 8u) + table_lane));
  return v;
}

// Loads the 16 code bits that each of the batch's workers m0 .. m0 + 4 kG4 - 1 holds for the eight
// coordinates of oct o, and adds their decoded values to q (Eq. SynQ_t before the division by M).
// lut_lane is the shared-memory address of the lane's copy of the batch's first table.  kLast: the batch holds the last
// worker group, the only one that can be short of workers.  Returns true if a code value 3 was met.
template <int kG4, bool kLast>
__device__ __forceinline__ bool decode_batch(const uint8_t* __restrict__ codes8, uint32_t row_bytes,
                                             uint64_t o, uint32_t m0, uint32_t M, uint32_t lut_lane,
                                             double (&q)[8]) {
  uint32_t c[4 * kG4];
  // row_bytes fits 32 bits (the launcher checks), so a worker's address is one widening multiply-add
  const uint8_t* p = codes8 + static_cast<uint64_t>(m0) * row_bytes + 2 * o;
#pragma unroll
  for (int m = 0; m < 4 * kG4; ++m)
    c[m] = (!kLast || m < 4 * (kG4 - 1) || m0 + m < M)
               ? __ldg(reinterpret_cast<const uint16_t*>(p + static_cast<uint64_t>(row_bytes) * static_cast<uint32_t>(m)))
               : 0u;
  uint32_t lo[kG4], hi[kG4], threes = 0;
#pragma unroll
  for (int G = 0; G < kG4; ++G) {
    // byte k of lo (hi) = worker 4G+k's codes of coordinates 0..3 (4..7)
    const uint32_t ab = __byte_perm(c[4 * G], c[4 * G + 1], 0x5140);
    const uint32_t cd = __byte_perm(c[4 * G + 2], c[4 * G + 3], 0x5140);
    lo[G] = __byte_perm(ab, cd, 0x5410);
    hi[G] = __byte_perm(ab, cd, 0x7632);
    threes |= (lo[G] & (lo[G] >> 1)) | (hi[G] & (hi[G] >> 1));
  }
  const bool bad = (threes & 0x55555555u) != 0u;
  if (bad) {  // rare: clear the fields that hold 3 before they are used as digits
#pragma unroll
    for (int G = 0; G < kG4; ++G) {
      lo[G] &= ~((lo[G] & (lo[G] >> 1) & 0x55555555u) * 3u);
      hi[G] &= ~((hi[G] & (hi[G] >> 1) & 0x55555555u) * 3u);
    }
  }
  // A word masked down to one field per byte holds four digits; in its product with the weights the
  // top byte collects byte0 + 3 byte1 + 9 byte2 + 27 byte3 <= 80: the other partial products fall
  // below bit 24, in disjoint fields, or leave the 32 bits.
  constexpr uint32_t kRadix3 = 0x0103091Bu;
#pragma unroll
  for (int G = 0; G < kG4; ++G) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const uint32_t il = (((lo[G] >> (2 * j)) & 0x03030303u) * kRadix3) >> 24;
      const uint32_t ih = (((hi[G] >> (2 * j)) & 0x03030303u) * kRadix3) >> 24;
      q[j] += lut3_entry(lut_lane + G * (kLut3Entries * kLut3Lanes * 8), il);
      q[4 + j] += lut3_entry(lut_lane + G * (kLut3Entries * kLut3Lanes * 8), ih);
    }
  }
  return bad;
}

__device__ __forceinline__ void prefetch_l2(const void* p) {
  asm volatile("prefetch.global.L2 [%0];" ::"l"(p));
}
// One request for a run of bytes (16-byte aligned, a multiple of 16 long) to be brought into L2: it holds no
// register and no shared memory while it is in flight.
__device__ __forceinline__ void prefetch_l2_bulk(const void* p, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}

// Two CTAs of kWideThreads threads per SM.  The workers are decoded in batches of 16 (their code bits
// are the only loads in flight then); the state of the eight coordinates is requested into L2 first and
// loaded once the average is known, so that it does not hold registers during the decode.
template <int kRule, int kM4>
__global__ void __launch_bounds__(kWideThreads, 2)
decode_update_wide_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ scales, uint64_t d,
                          uint32_t M, double inv_m, float* __restrict__ x, float* __restrict__ h,
                          float* __restrict__ z, StepScalars sc, unsigned int* __restrict__ status) {
  extern __shared__ double sm_lut[];
  chain_wait();  // scales and codes come from the launch before this one
  chain_trigger();
  build_decode_lut3(sm_lut, scales, M);
  const uint32_t lut_lane =
      static_cast<uint32_t>(__cvta_generic_to_shared(sm_lut + (threadIdx.x & (kLut3Lanes - 1))));
  const uint8_t* codes8 = reinterpret_cast<const uint8_t*>(codes);
  const uint32_t row_bytes = static_cast<uint32_t>(((d + 15) >> 4) * 4);
  const uint64_t octs = (d + 7) >> 3, full = d >> 3;
  const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kWideThreads;
  constexpr int kBatch = 4;                         // worker groups per batch
  constexpr int kWholeBatches = (kM4 - 1) / kBatch;  // batches before the last one
  bool bad = false;
  for (uint64_t o = static_cast<uint64_t>(blockIdx.x) * kWideThreads + threadIdx.x; o < octs; o += stride) {
    const bool whole = o < full;
    float* ap = (kRule == 0 ? x : z) + 8 * o;  // x for QCMD (read and written), z for QRDA
    if (kRule != 2 && whole) {
      prefetch_l2(h + 8 * o);
      prefetch_l2(ap);
    }
    double q[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) q[i] = 0.0;
#pragma unroll
    for (int b = 0; b < kWholeBatches; ++b)
      bad |= decode_batch<kBatch, false>(codes8, row_bytes, o, 4 * kBatch * b, M,
                                         lut_lane + b * (kBatch * kLut3Entries * kLut3Lanes * 8), q);
    bad |= decode_batch<kM4 - kBatch * kWholeBatches, true>(
        codes8, row_bytes, o, 4 * kBatch * kWholeBatches, M,
        lut_lane + kWholeBatches * (kBatch * kLut3Entries * kLut3Lanes * 8), q);
    float qf[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) qf[i] = static_cast<float>(q[i] * inv_m);
    if (whole) {
      if (kRule == 2) {
        *reinterpret_cast<float4*>(x + 8 * o) = make_float4(qf[0], qf[1], qf[2], qf[3]);
        *reinterpret_cast<float4*>(x + 8 * o + 4) = make_float4(qf[4], qf[5], qf[6], qf[7]);
        continue;
      }
      float4 h0 = *reinterpret_cast<const float4*>(h + 8 * o);
      float4 h1 = *reinterpret_cast<const float4*>(h + 8 * o + 4);
      float4 a0 = *reinterpret_cast<const float4*>(ap);
      float4 a1 = *reinterpret_cast<const float4*>(ap + 4);
      if (kRule == 0) {
        cmd_update(qf[0], a0.x, h0.x, sc), cmd_update(qf[1], a0.y, h0.y, sc);
        cmd_update(qf[2], a0.z, h0.z, sc), cmd_update(qf[3], a0.w, h0.w, sc);
        cmd_update(qf[4], a1.x, h1.x, sc), cmd_update(qf[5], a1.y, h1.y, sc);
        cmd_update(qf[6], a1.z, h1.z, sc), cmd_update(qf[7], a1.w, h1.w, sc);
        *reinterpret_cast<float4*>(x + 8 * o) = a0;
        *reinterpret_cast<float4*>(x + 8 * o + 4) = a1;
      } else {
        float4 x0, x1;
        rda_update(qf[0], x0.x, h0.x, a0.x, sc), rda_update(qf[1], x0.y, h0.y, a0.y, sc);
        rda_update(qf[2], x0.z, h0.z, a0.z, sc), rda_update(qf[3], x0.w, h0.w, a0.w, sc);
        rda_update(qf[4], x1.x, h1.x, a1.x, sc), rda_update(qf[5], x1.y, h1.y, a1.y, sc);
        rda_update(qf[6], x1.z, h1.z, a1.z, sc), rda_update(qf[7], x1.w, h1.w, a1.w, sc);
        *reinterpret_cast<float4*>(z + 8 * o) = a0;
        *reinterpret_cast<float4*>(z + 8 * o + 4) = a1;
        *reinterpret_cast<float4*>(x + 8 * o) = x0;
        *reinterpret_cast<float4*>(x + 8 * o + 4) = x1;
      }
      *reinterpret_cast<float4*>(h + 8 * o) = h0;
      *reinterpret_cast<float4*>(h + 8 * o + 4) = h1;
    } else {  // ragged tail: d % 8 coordinates
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const uint64_t i = 8 * o + e;
        if (i >= d) break;
        const float qi = qf[e];
        if (kRule == 2) {
          x[i] = qi;
          continue;
        }
        float xi = (kRule == 0) ? x[i] : 0.f, hi = h[i];
        if (kRule == 0) {
          cmd_update(qi, xi, hi, sc);
        } else {
          float zi = z[i];
          rda_update(qi, xi, hi, zi, sc);
          z[i] = zi;
        }
        x[i] = xi;
        h[i] = hi;
      }
    }
  }
  if (bad) atomicOr(status, kFlagBadCode);
}

// ------------------------------------------------------------------ pass C, update from a dense q
template <int kRule>
__global__ void __launch_bounds__(kThreads)
dense_update_kernel(const float* __restrict__ q, uint64_t d, float* __restrict__ x,
                    float* __restrict__ h, float* __restrict__ z, StepScalars sc) {
  const uint64_t full = d >> 2;
  const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;
  const uint64_t first = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
  for (uint64_t grp = first; grp < full; grp += stride) {
    const float4 qv = __ldg(reinterpret_cast<const float4*>(q) + grp);
    float4 hv = *reinterpret_cast<const float4*>(h + 4 * grp);
    float4 xv, zv;
    if (kRule == 0) {
      xv = *reinterpret_cast<const float4*>(x + 4 * grp);
      cmd_update(qv.x, xv.x, hv.x, sc);
      cmd_update(qv.y, xv.y, hv.y, sc);
      cmd_update(qv.z, xv.z, hv.z, sc);
      cmd_update(qv.w, xv.w, hv.w, sc);
    } else {
      zv = *reinterpret_cast<const float4*>(z + 4 * grp);
      rda_update(qv.x, xv.x, hv.x, zv.x, sc);
      rda_update(qv.y, xv.y, hv.y, zv.y, sc);
      rda_update(qv.z, xv.z, hv.z, zv.z, sc);
      rda_update(qv.w, xv.w, hv.w, zv.w, sc);
      *reinterpret_cast<float4*>(z + 4 * grp) = zv;
    }
    *reinterpret_cast<float4*>(h + 4 * grp) = hv;
    *reinterpret_cast<float4*>(x + 4 * grp) = xv;
  }
  if (first == 0) {
    for (uint64_t i = 4 * full; i < d; ++i) {
      float xi = (kRule == 0) ? x[i] : 0.f, hi = h[i];
      if (kRule == 0) {
        cmd_update(q[i], xi, hi, sc);
      } else {
        float zi = z[i];
        rda_update(q[i], xi, hi, zi, sc);
        z[i] = zi;
      }
      x[i] = xi;
      h[i] = hi;
    }
  }
}

// ------------------------------------------------------------------ pass C without quantization
// q_t = plain mean of the M fp32 gradients (32-bit CMD / RDA adagrad): per coordinate the M values
// are read once, summed in fp64 in worker order, scaled by 1/M and rounded to fp32; then the same
// accumulator and update as above.  A thread owns four coordinates; eight rows are in flight at a time.
template <int kRule>
__global__ void __launch_bounds__(kThreads)
mean_update_kernel(const float* __restrict__ g, uint64_t d, uint64_t ld, uint32_t M, double inv_m,
                   float* __restrict__ x, float* __restrict__ h, float* __restrict__ z, StepScalars sc,
                   unsigned int* __restrict__ status) {
  const uint64_t full = d >> 2;
  const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;
  const uint64_t first = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
  bool nonfinite = false;
  for (uint64_t grp = first; grp < full; grp += stride) {
    float4 hv = *reinterpret_cast<const float4*>(h + 4 * grp);
    float4 av = *reinterpret_cast<const float4*>((kRule == 0 ? x : z) + 4 * grp);
    const float* p = g + 4 * grp;
    double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0;
    uint32_t m = 0;
    for (; m + 8 <= M; m += 8) {
      float4 v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) v[k] = load_f4(p + static_cast<uint64_t>(m + k) * ld);
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        a0 += static_cast<double>(v[k].x);
        a1 += static_cast<double>(v[k].y);
        a2 += static_cast<double>(v[k].z);
        a3 += static_cast<double>(v[k].w);
      }
    }
    for (; m < M; ++m) {
      const float4 v = load_f4(p + static_cast<uint64_t>(m) * ld);
      a0 += static_cast<double>(v.x);
      a1 += static_cast<double>(v.y);
      a2 += static_cast<double>(v.z);
      a3 += static_cast<double>(v.w);
    }
    const float4 q = make_float4(static_cast<float>(a0 * inv_m), static_cast<float>(a1 * inv_m),
                                 static_cast<float>(a2 * inv_m), static_cast<float>(a3 * inv_m));
    nonfinite |= !(fabsf(q.x) <= 3.402823466e38f) | !(fabsf(q.y) <= 3.402823466e38f) |
                 !(fabsf(q.z) <= 3.402823466e38f) | !(fabsf(q.w) <= 3.402823466e38f);
    if (kRule == 0) {
      cmd_update(q.x, av.x, hv.x, sc);
      cmd_update(q.y, av.y, hv.y, sc);
      cmd_update(q.z, av.z, hv.z, sc);
      cmd_update(q.w, av.w, hv.w, sc);
      *reinterpret_cast<float4*>(x + 4 * grp) = av;
    } else {
      float4 xv;
      rda_update(q.x, xv.x, hv.x, av.x, sc);
      rda_update(q.y, xv.y, hv.y, av.y, sc);
      rda_update(q.z, xv.z, hv.z, av.z, sc);
      rda_update(q.w, xv.w, hv.w, av.w, sc);
      *reinterpret_cast<float4*>(z + 4 * grp) = av;
      *reinterpret_cast<float4*>(x + 4 * grp) = xv;
    }
    *reinterpret_cast<float4*>(h + 4 * grp) = hv;
  }
  if (first == 0) {  // ragged tail: d % 4 coordinates
    for (uint64_t i = 4 * full; i < d; ++i) {
      double acc = 0.0;
      for (uint32_t m = 0; m < M; ++m) acc += static_cast<double>(g[static_cast<uint64_t>(m) * ld + i]);
      const float q = static_cast<float>(acc * inv_m);
      nonfinite |= !(fabsf(q) <= 3.402823466e38f);
      float xi = (kRule == 0) ? x[i] : 0.f, hi = h[i];
      if (kRule == 0) {
        cmd_update(q, xi, hi, sc);
      } else {
        float zi = z[i];
        rda_update(q, xi, hi, zi, sc);
        z[i] = zi;
      }
      x[i] = xi;
      h[i] = hi;
    }
  }
  if (nonfinite) atomicOr(status, kFlagNonFinite);
}

// ------------------------------------------------------------------ server row: q = Q(average)
// Double quantization (Algorithm 1, "Quantize the aggregated gradient"): the averaged gradient is
// quantized again with the same Q.  The average is never stored: these kernels rebuild it from the
// workers' code bytes, tile by tile, in the same 4 x 1024 tile geometry as a worker's gradient, so
// its threshold and scale come from the same fixed-order sums.  The row is cut into up to
// kRowChunks chunks; the last CTA combines their partials with a pairwise tree over 8 blocks of
// 1024 slots, which is the pairwise tree over all slots.

// The thread's four float4 of tile k of the averaged gradient; coordinates >= d are +0.0.
__device__ __forceinline__ void decode_tile(const uint8_t* __restrict__ codes8, uint64_t row_bytes,
                                            const double* lut, uint32_t workers, double inv_m, uint64_t d,
                                            uint32_t k, int j, float4 (&v)[kTileRows], uint32_t& bad) {
#pragma unroll
  for (int r = 0; r < kTileRows; ++r) {
    const uint64_t grp = static_cast<uint64_t>(k) * (kTile / 4) + r * (kTileCols / 4) + j;
    const uint64_t i0 = 4 * grp;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 < d) {
      t = decode_group<0, 1>(codes8, row_bytes, lut, workers, inv_m, grp, bad);
      if (i0 + 1 >= d) t.y = 0.f;
      if (i0 + 2 >= d) t.z = 0.f;
      if (i0 + 3 >= d) t.w = 0.f;
    }
    v[r] = t;
  }
}

// Pairwise tree over up to kRowChunks = 8 * 1024 partial slots; all threads call, result in thread 0.
__device__ __forceinline__ double block_chunk_tree(const double* part, uint32_t chunks, double* sm8) {
  const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t base = warp * kMaxChunks;
  const double v = warp_chunk_tree(part + base, chunks > base ? chunks - base : 0u, lane);
  __syncthreads();
  if (lane == 0) sm8[warp] = v;
  __syncthreads();
  double r = 0.0;
  if (threadIdx.x == 0) r = ((sm8[0] + sm8[1]) + (sm8[2] + sm8[3])) + ((sm8[4] + sm8[5]) + (sm8[6] + sm8[7]));
  return r;
}

__global__ void __launch_bounds__(kThreads, 4)
avg_abs_sum_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ scales, uint32_t workers,
                   double inv_m, Geometry geo, float coef, Workspace ws, float* __restrict__ threshold_out,
                   const unsigned long long* __restrict__ denom) {
  extern __shared__ double sm_lut[];
  __shared__ ChunkSumStorage sm_sum;
  __shared__ double sm8[kThreads / 32];
  __shared__ bool sm_last;
  build_decode_lut<1>(sm_lut, scales, workers);
  const int j = threadIdx.x;
  const uint8_t* codes8 = reinterpret_cast<const uint8_t*>(codes);
  const uint64_t row_bytes = ((geo.d + 15) >> 4) * 4;
  ChunkSum chunk_sum(&sm_sum);
  uint32_t bad = 0;
  for (uint32_t c = blockIdx.x; c < geo.chunks; c += gridDim.x) {
    const uint32_t k0 = c * geo.group;
    const uint32_t k1 = min(k0 + geo.group, geo.tiles);
    for (uint32_t k = k0; k < k1; ++k) {
      float4 v[kTileRows];
      decode_tile(codes8, row_bytes, sm_lut, workers, inv_m, geo.d, k, j, v, bad);
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
    const double total = chunk_sum.finish(geo.log2_group);
    if (j == 0) ws.part_sum[c] = total;
  }
  if (bad) atomicOr(ws.status, kFlagBadCode);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  const double total = block_chunk_tree(ws.part_sum, geo.chunks, sm8);
  if (j == 0) {
    const unsigned long long n = denom ? denom[0] : geo.d;
    const float delta = n ? static_cast<float>((static_cast<double>(coef) * total) / static_cast<double>(n)) : 0.f;
    ws.thresholds[0] = delta;
    if (threshold_out) threshold_out[0] = delta;
    *ws.ticket = 0u;
  }
}

__global__ void __launch_bounds__(kThreads, 4)
avg_abs_max_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ scales, uint32_t workers,
                   double inv_m, Geometry geo, Workspace ws) {
  extern __shared__ double sm_lut[];
  __shared__ uint32_t sm_warp[kThreads / 32];
  __shared__ bool sm_last;
  build_decode_lut<1>(sm_lut, scales, workers);
  const int j = threadIdx.x;
  const uint8_t* codes8 = reinterpret_cast<const uint8_t*>(codes);
  const uint64_t row_bytes = ((geo.d + 15) >> 4) * 4;
  uint32_t bad = 0, best = 0u;
  for (uint32_t c = blockIdx.x; c < geo.chunks; c += gridDim.x) {
    const uint32_t k0 = c * geo.group;
    const uint32_t k1 = min(k0 + geo.group, geo.tiles);
    for (uint32_t k = k0; k < k1; ++k) {
      float4 v[kTileRows];
      decode_tile(codes8, row_bytes, sm_lut, workers, inv_m, geo.d, k, j, v, bad);
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        best = max(best, __float_as_uint(fabsf(v[r].x)));
        best = max(best, __float_as_uint(fabsf(v[r].y)));
        best = max(best, __float_as_uint(fabsf(v[r].z)));
        best = max(best, __float_as_uint(fabsf(v[r].w)));
      }
    }
  }
  // the maximum is order-free: one partial per CTA
  best = __reduce_max_sync(0xffffffffu, best);
  if ((j & 31) == 0) sm_warp[j >> 5] = best;
  __syncthreads();
  if (j == 0) {
    uint32_t bmax = sm_warp[0];
#pragma unroll
    for (int w = 1; w < kThreads / 32; ++w) bmax = max(bmax, sm_warp[w]);
    ws.part_max[blockIdx.x] = bmax;
  }
  if (bad) atomicOr(ws.status, kFlagBadCode);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  uint32_t bmax = 0u;
  for (uint32_t idx = j; idx < gridDim.x; idx += kThreads) bmax = max(bmax, __ldcg(ws.part_max + idx));
  bmax = __reduce_max_sync(0xffffffffu, bmax);
  __syncthreads();
  if ((j & 31) == 0) sm_warp[j >> 5] = bmax;
  __syncthreads();
  if (j == 0) {
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) bmax = max(bmax, sm_warp[w]);
    ws.scales[0] = __uint_as_float(bmax);
    ws.thresholds[0] = 0.f;
    *ws.ticket = 0u;
  }
}

// kStochastic = false: Q_Delta with ws.thresholds[0]; true: unbiased ternary with ws.scales[0] and the
// Philox stream of domain 1 (worker field 0).
template <bool kStochastic>
__global__ void __launch_bounds__(kThreads, 4)
avg_codes_kernel(const uint32_t* __restrict__ codes, const float* __restrict__ scales, uint32_t workers,
                 double inv_m, Geometry geo, uint64_t seed, uint64_t t, Workspace ws,
                 uint32_t* __restrict__ qcodes, float* __restrict__ scale_out,
                 unsigned long long* __restrict__ count_out) {
  extern __shared__ double sm_lut[];
  __shared__ ChunkSumStorage sm_sum;
  __shared__ double sm8[kThreads / 32];
  __shared__ uint32_t sm_cnt[kThreads / 32];
  __shared__ bool sm_last;
  build_decode_lut<1>(sm_lut, scales, workers);
  const int j = threadIdx.x;
  const uint8_t* codes8 = reinterpret_cast<const uint8_t*>(codes);
  uint8_t* qcodes8 = reinterpret_cast<uint8_t*>(qcodes);
  const uint64_t row_bytes = ((geo.d + 15) >> 4) * 4;
  const uint32_t full_tiles = static_cast<uint32_t>(geo.d / kTile);
  const float delta = ws.thresholds[0], ndelta = -delta, smax = ws.scales[0];
  const uint32_t key0 = static_cast<uint32_t>(seed), key1 = static_cast<uint32_t>(seed >> 32);
  const uint32_t t_lo = static_cast<uint32_t>(t), t_hi = static_cast<uint32_t>(t >> 32);
  ChunkSum chunk_sum(&sm_sum);
  uint32_t bad = 0;
  for (uint32_t c = blockIdx.x; c < geo.chunks; c += gridDim.x) {
    const uint32_t k0 = c * geo.group;
    const uint32_t k1 = min(k0 + geo.group, geo.tiles);
    float cntf = 0.f;
    for (uint32_t k = k0; k < k1; ++k) {
      float4 v[kTileRows];
      decode_tile(codes8, row_bytes, sm_lut, workers, inv_m, geo.d, k, j, v, bad);
      double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
      uint32_t bytes[kTileRows];
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        const float4 q = v[r];
        float px, nx, py, ny, pz, nz, pw, nw;
        if (!kStochastic) {
          px = q.x > delta ? 1.f : 0.f, nx = q.x < ndelta ? 1.f : 0.f;
          py = q.y > delta ? 1.f : 0.f, ny = q.y < ndelta ? 1.f : 0.f;
          pz = q.z > delta ? 1.f : 0.f, nz = q.z < ndelta ? 1.f : 0.f;
          pw = q.w > delta ? 1.f : 0.f, nw = q.w < ndelta ? 1.f : 0.f;
        } else {
          const uint32_t blk = k * (kTile / 4) + r * (kTileCols / 4) + j;
          const uint4 w = philox4x32_10(make_uint4(blk, 1u << 16, t_lo, t_hi), key0, key1);
          const CodeBits bx = split_code(q.x, philox_uniform(w.x) < __fdiv_rn(fabsf(q.x), smax));
          const CodeBits by = split_code(q.y, philox_uniform(w.y) < __fdiv_rn(fabsf(q.y), smax));
          const CodeBits bz = split_code(q.z, philox_uniform(w.z) < __fdiv_rn(fabsf(q.z), smax));
          const CodeBits bw = split_code(q.w, philox_uniform(w.w) < __fdiv_rn(fabsf(q.w), smax));
          px = bx.pos, nx = bx.neg, py = by.pos, ny = by.neg, pz = bz.pos, nz = bz.neg, pw = bw.pos, nw = bw.neg;
        }
        const float kx = px + nx, ky = py + ny, kz = pz + nz, kw = pw + nw;
        if (!kStochastic) {
          cx += static_cast<double>(fabsf(q.x) * kx);
          cy += static_cast<double>(fabsf(q.y) * ky);
          cz += static_cast<double>(fabsf(q.z) * kz);
          cw += static_cast<double>(fabsf(q.w) * kw);
        }
        cntf += (kx + ky) + (kz + kw);
        bytes[r] = pack4({px, nx}, {py, ny}, {pz, nz}, {pw, nw});
      }
      store_code_bytes(qcodes8, k, j, k < full_tiles, row_bytes, bytes);
      if (!kStochastic) chunk_sum.add_tile((cx + cy) + (cz + cw));
    }
    double picked = 0.0;
    if (!kStochastic) picked = chunk_sum.finish(geo.log2_group);
    const unsigned long long total = block_count(static_cast<uint32_t>(cntf), sm_cnt);
    if (j == 0) {
      ws.part_sum[c] = picked;
      ws.part_cnt[c] = total;
    }
  }
  if (bad) atomicOr(ws.status, kFlagBadCode);
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  unsigned long long n = 0;
  for (uint32_t idx = j; idx < geo.chunks; idx += kThreads) n += __ldcg(ws.part_cnt + idx);
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) n += __shfl_xor_sync(0xffffffffu, n, s);
  __shared__ unsigned long long sm_n[kThreads / 32];
  if ((j & 31) == 0) sm_n[j >> 5] = n;
  const double picked = kStochastic ? 0.0 : block_chunk_tree(ws.part_sum, geo.chunks, sm8);
  __syncthreads();
  if (j == 0) {
    n = 0;
#pragma unroll
    for (int w = 0; w < kThreads / 32; ++w) n += sm_n[w];
    const float scale = kStochastic ? smax : (n ? static_cast<float>(picked / static_cast<double>(n)) : 0.f);
    ws.scales[0] = scale;
    ws.counts[0] = n;
    if (scale_out) scale_out[0] = scale;
    if (count_out) count_out[0] = n;
    *ws.ticket = 0u;
  }
}

// ------------------------------------------------------------------ sparse selection
// Indicator of one coordinate of one worker (Section 3.2): x != 0, or the worker's local trial update
// with its own gradient leaves the coordinate non-zero.  Where x != 0 the bit is set whatever the trial
// gives; where x == 0 the closed form of the trial update is non-zero iff
//   QCMD: |g| > lambda          (H_hat = delta + sqrt(h + g*g) > 0 scales both sides and drops out)
//   QRDA: |z + g| > lambda*t    (hz = z; one correctly rounded addition, no fused multiply-add)
// so one fp32 comparison decides the bit and it does not depend on who computes it.
template <int kRule>
__device__ __forceinline__ bool selects(float g, float x, float hz, const SelectScalars& sc) {
  const bool moved = kRule == 0 ? fabsf(g) > sc.lambda : fabsf(__fadd_rn(hz, g)) > sc.lambda_t;
  return (x != 0.f) || moved;
}

// A thread's four float4 of tile k of a state vector of exactly d floats (no padding to read into).
__device__ __forceinline__ void load_state_tile(const float* __restrict__ v, uint64_t d, uint32_t k, int j,
                                                bool whole, float4 (&out)[kTileRows]) {
  if (whole) {  // the tile lies inside [0, d): no bounds tests
#pragma unroll
    for (int r = 0; r < kTileRows; ++r)
      out[r] = load_f4(v + static_cast<uint64_t>(k) * kTile + r * kTileCols + 4 * j);
    return;
  }
#pragma unroll
  for (int r = 0; r < kTileRows; ++r) {
    const uint64_t i0 = static_cast<uint64_t>(k) * kTile + r * kTileCols + 4 * j;
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i0 + 4 <= d) {
      t = load_f4(v + i0);
    } else if (i0 < d) {
      t.x = v[i0];
      if (i0 + 1 < d) t.y = v[i0 + 1];
      if (i0 + 2 < d) t.z = v[i0 + 2];
    }
    out[r] = t;
  }
}

// Pass A with selection: writes each worker's indicator bits and reduces, over the selected
// coordinates only, the sum of |g| (threshold quantizer: Delta_m = coef * sum / k_m) or the maximum
// (stochastic quantizer), and k_m.
// One CTA takes one chunk of tiles for ALL workers: per tile it loads x and h (or z) once into
// registers and walks the M gradient tiles (the next worker's loads in flight), so the state is read
// once per coordinate, not once per worker.  Every worker keeps its own fixed-order sum: the same
// column sums, warp butterfly, 8-warp combine and pairwise stack over tiles as in abs_sum_kernel,
// with the cross-warp combine batched over kSelectBatch tiles.
constexpr int kSelectBatch = 8;
constexpr int kSelectDoublesPerWorker = kSelectBatch * (kThreads / 32) + kSelectBatch + 32;

__host__ __device__ inline size_t select_smem_bytes(uint32_t M) {
  return static_cast<size_t>(M) * (kSelectDoublesPerWorker * sizeof(double) + 2 * sizeof(uint32_t));
}

template <int kRule, bool kStochastic>
__global__ void __launch_bounds__(kThreads, kSelectCtasPerSm)
select_stats_kernel(const float* __restrict__ g, Geometry geo, const float* __restrict__ x,
                    const float* __restrict__ hz, SelectScalars sc, float coef, Workspace ws,
                    uint32_t* __restrict__ indicators, float* __restrict__ thresholds_out,
                    unsigned long long* __restrict__ selected_out) {
  extern __shared__ double sm_dyn[];
  __shared__ bool sm_last;
  const uint32_t M = geo.M;
  double* warp_sums = sm_dyn;                                        // [M][kSelectBatch][8]
  double* tile_sums = warp_sums + M * kSelectBatch * (kThreads / 32);  // [M][kSelectBatch]
  double* stacks = tile_sums + M * kSelectBatch;                      // [M][32]
  uint32_t* sm_cnt = reinterpret_cast<uint32_t*>(stacks + M * 32);     // [M] selected in this chunk
  uint32_t* sm_max = sm_cnt + M;                                      // [M] max |g| over the selected
  const int j = threadIdx.x, warp = j >> 5, lane = j & 31;
  const uint64_t ind_words = (geo.d + 31) >> 5;
  for (uint32_t c = blockIdx.x; c < geo.chunks; c += gridDim.x) {
    const uint32_t k0 = c * geo.group;
    const uint32_t k1 = min(k0 + geo.group, geo.tiles);
    for (uint32_t m = j; m < 2 * M; m += kThreads) sm_cnt[m] = 0u;  // counts and maxima
    __syncthreads();
    uint32_t pending = 0, pushed = 0;
    // The chunk is one stream of gradient tiles, (tile k, worker 0..M-1), (tile k+1, worker 0..M-1), ...:
    // the next one is always in flight.  The state of a tile is read at its start.
    // Of x only "non-zero" is kept, folded into the level each coordinate is compared with: -1 where
    // x != 0 (every magnitude exceeds it), lambda (QRDA: lambda t) elsewhere.  The comparison is
    // "greater or unordered": a NaN is marked, enters the sums and is reported.
    float4 ga[kTileRows], gb[kTileRows], level[kTileRows], zc[kTileRows];
    bool a_cur = true;
    auto whole_tile = [&](uint32_t k) { return static_cast<uint64_t>(k + 1) * kTile <= geo.d; };
    const float base_level = kRule == 0 ? sc.lambda : sc.lambda_t;
    load_tile(g, static_cast<uint64_t>(k0) * kTile, geo.d, j, ga);
    for (uint32_t k = k0; k < k1; ++k) {
      const uint64_t tile_base = static_cast<uint64_t>(k) * kTile;
      const bool whole = whole_tile(k);
      load_state_tile(x, geo.d, k, j, whole, level);
      if (kRule == 1) load_state_tile(hz, geo.d, k, j, whole, zc);
#pragma unroll
      for (int r = 0; r < kTileRows; ++r) {
        level[r].x = level[r].x != 0.f ? -1.f : base_level;
        level[r].y = level[r].y != 0.f ? -1.f : base_level;
        level[r].z = level[r].z != 0.f ? -1.f : base_level;
        level[r].w = level[r].w != 0.f ? -1.f : base_level;
      }
      // Two adjacent threads share an indicator byte and the even one writes it.  A tile that is not whole
      // may reach past the row's last indicator word: those bytes are not written (the bits below d's word
      // boundary that lie at or past d come out 0, since g, x and z read as +0.0 there).
      const uint64_t byte0 = (tile_base >> 3) + (j >> 1);
      uint32_t rows_written = kTileRows;
      if (!whole) {
        const uint64_t left = ind_words * 4 > byte0 ? (ind_words * 4 - byte0 + kTileCols / 8 - 1) / (kTileCols / 8) : 0;
        rows_written = left < kTileRows ? static_cast<uint32_t>(left) : kTileRows;
      }
      if (j & 1) rows_written = 0u;
      // One worker's share of this tile: indicator bits, selected |g| into the fixed-order sum.
      auto worker_tile = [&](const float4 (&gv)[kTileRows], uint32_t m) {
        uint8_t* ind8 = reinterpret_cast<uint8_t*>(indicators + static_cast<uint64_t>(m) * ind_words) + byte0;
        double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
        uint32_t cnt = 0u, best = 0u;
#pragma unroll
        for (int r = 0; r < kTileRows; ++r) {
          const float4 gr = gv[r];
          float dx = gr.x, dy = gr.y, dz = gr.z, dw = gr.w;
          if (kRule == 1) {
            dx = __fadd_rn(zc[r].x, gr.x), dy = __fadd_rn(zc[r].y, gr.y);
            dz = __fadd_rn(zc[r].z, gr.z), dw = __fadd_rn(zc[r].w, gr.w);
          }
          const float px = !(fabsf(dx) <= level[r].x) ? 1.f : 0.f, py = !(fabsf(dy) <= level[r].y) ? 1.f : 0.f;
          const float pz = !(fabsf(dz) <= level[r].z) ? 1.f : 0.f, pw = !(fabsf(dw) <= level[r].w) ? 1.f : 0.f;
          const float sx = fabsf(gr.x) * px, sy = fabsf(gr.y) * py, sz = fabsf(gr.z) * pz, sw = fabsf(gr.w) * pw;
          if (!kStochastic) {
            cx += static_cast<double>(sx);
            cy += static_cast<double>(sy);
            cz += static_cast<double>(sz);
            cw += static_cast<double>(sw);
          } else {
            best = max(max(best, __float_as_uint(sx)), __float_as_uint(sy));
            best = max(max(best, __float_as_uint(sz)), __float_as_uint(sw));
          }
          const uint32_t nib = static_cast<uint32_t>(fmaf(8.f, pw, fmaf(4.f, pz, fmaf(2.f, py, px))));
          cnt += __popc(nib);
          const uint32_t upper = __shfl_down_sync(0xffffffffu, nib, 1);
          if (static_cast<uint32_t>(r) < rows_written) ind8[r * (kTileCols / 8)] = static_cast<uint8_t>(nib | (upper << 4));
        }
        if (!kStochastic) {
          const double v = warp_pair_tree((cx + cy) + (cz + cw));
          if (lane == 0) warp_sums[(m * kSelectBatch + pending) * (kThreads / 32) + warp] = v;
        } else {
          best = __reduce_max_sync(0xffffffffu, best);
          if (lane == 0 && best) atomicMax(&sm_max[m], best);
        }
        cnt = __reduce_add_sync(0xffffffffu, cnt);
        if (lane == 0 && cnt) atomicAdd(&sm_cnt[m], cnt);
      };
      for (uint32_t m = 0; m < M; ++m) {
        auto prefetch = [&](float4 (&nxt)[kTileRows]) {
          if (m + 1 < M) {
            load_tile(g + static_cast<uint64_t>(m + 1) * geo.ld, tile_base, geo.d, j, nxt);
          } else if (k + 1 < k1) {
            load_tile(g, tile_base + kTile, geo.d, j, nxt);
          }
        };
        if (a_cur) {
          prefetch(gb);
          worker_tile(ga, m);
        } else {
          prefetch(ga);
          worker_tile(gb, m);
        }
        a_cur = !a_cur;
      }
      ++pending;
      if (!kStochastic && (pending == kSelectBatch || k + 1 == k1)) {
        __syncthreads();
        for (uint32_t e = j; e < M * pending; e += kThreads) {  // (worker, tile): combine the 8 warps
          const uint32_t wm = e / pending, p = e - wm * pending;
          const double* a = warp_sums + (wm * kSelectBatch + p) * (kThreads / 32);
          tile_sums[wm * kSelectBatch + p] = ((a[0] + a[1]) + (a[2] + a[3])) + ((a[4] + a[5]) + (a[6] + a[7]));
        }
        __syncthreads();
        for (uint32_t wm = j; wm < M; wm += kThreads)  // one thread per worker pushes its tiles, in order
          for (uint32_t p = 0; p < pending; ++p) tile_push(stacks + wm * 32, pushed + p, tile_sums[wm * kSelectBatch + p]);
        pushed += pending;
        pending = 0;
      }
    }
    __syncthreads();
    for (uint32_t wm = j; wm < M; wm += kThreads) {
      const uint64_t p = static_cast<uint64_t>(wm) * kRowChunks + c;
      ws.part_sum[p] = kStochastic ? 0.0 : tile_fold(stacks + wm * 32, pushed, geo.log2_group);
      ws.part_cnt[p] = sm_cnt[wm];
      ws.part_max[p] = sm_max[wm];
    }
    __syncthreads();
  }
  __threadfence();  // every thread that wrote partials publishes them before the CTA takes its ticket
  __syncthreads();
  if (!grid_last_cta(ws.ticket, &sm_last)) return;
  for (uint32_t m = warp; m < geo.M; m += kThreads / 32) {
    unsigned long long n = 0;
    uint32_t bmax = 0u;
    for (uint32_t idx = lane; idx < geo.chunks; idx += 32) {
      n += __ldcg(ws.part_cnt + static_cast<uint64_t>(m) * kRowChunks + idx);
      if (kStochastic) bmax = max(bmax, __ldcg(ws.part_max + static_cast<uint64_t>(m) * kRowChunks + idx));
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) n += __shfl_xor_sync(0xffffffffu, n, s);
    double total = 0.0;
    if (!kStochastic) {  // pairwise tree over the worker's up to kRowChunks = 8 * kMaxChunks partials
      double blk[kRowChunks / kMaxChunks];
#pragma unroll 1
      for (uint32_t b = 0; b < kRowChunks / kMaxChunks; ++b) {
        const uint32_t base = b * kMaxChunks;
        blk[b] = warp_chunk_tree(ws.part_sum + static_cast<uint64_t>(m) * kRowChunks + base,
                                 geo.chunks > base ? geo.chunks - base : 0u, lane);
      }
      total = ((blk[0] + blk[1]) + (blk[2] + blk[3])) + ((blk[4] + blk[5]) + (blk[6] + blk[7]));
    }
    if (kStochastic) bmax = __reduce_max_sync(0xffffffffu, bmax);
    if (lane == 0) {
      ws.selected[m] = n;
      if (selected_out) selected_out[m] = n;
      if (!kStochastic) {
        const float delta = n ? static_cast<float>((static_cast<double>(coef) * total) / static_cast<double>(n)) : 0.f;
        ws.thresholds[m] = delta;
        if (thresholds_out) thresholds_out[m] = delta;
        if (!isfinite(total)) atomicOr(ws.status, kFlagNonFinite);
      } else {
        ws.scales[m] = __uint_as_float(bmax);
        ws.thresholds[m] = 0.f;
        if (thresholds_out) thresholds_out[m] = 0.f;
        if (bmax >= 0x7f800000u) atomicOr(ws.status, kFlagNonFinite);
      }
    }
  }
  if (j == 0) *ws.ticket = 0u;
}

// The synchronous indicator: "bitwise or" of the M workers' indicators, and how many bits it has.
__global__ void __launch_bounds__(kThreads)
indicator_or_kernel(const uint32_t* __restrict__ indicators, uint64_t words, uint32_t M,
                    uint32_t* __restrict__ isyn, unsigned long long* __restrict__ ksyn) {
  unsigned long long bits = 0;
  for (uint64_t w = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x; w < words;
       w += static_cast<uint64_t>(gridDim.x) * kThreads) {
    uint32_t acc = 0u;
    for (uint32_t m = 0; m < M; ++m) acc |= __ldg(indicators + m * words + w);
    isyn[w] = acc;
    bits += __popc(acc);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) bits += __shfl_xor_sync(0xffffffffu, bits, s);
  if ((threadIdx.x & 31) == 0 && bits) atomicAdd(ksyn, bits);
}

// ------------------------------------------------------------------ launchers
void query_launch_shape(LaunchShape* shape) {
  int dev = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&shape->sm_count, cudaDevAttrMultiProcessorCount, dev);
  int a = 0, b = 0;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&a, threshold_codes_kernel<false>, kThreads, 0);
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&b, dense_update_kernel<1>, kThreads, 0);
  shape->chained = false;
  shape->reduce_ctas_per_sm = a > 0 ? a : 1;
  shape->update_ctas_per_sm = b > 0 ? b : 1;
}

static unsigned reduce_grid(const Geometry& geo, const LaunchShape& shape) {
  const uint64_t items = static_cast<uint64_t>(geo.M) * geo.chunks;
  const uint64_t resident = static_cast<uint64_t>(shape.sm_count) * shape.reduce_ctas_per_sm;
  return static_cast<unsigned>(items < resident ? items : resident);
}

static unsigned update_grid(uint64_t d, const LaunchShape& shape) {
  const uint64_t groups = (d + 3) >> 2;
  const uint64_t ctas = (groups + kThreads - 1) / kThreads;
  const uint64_t resident = static_cast<uint64_t>(shape.sm_count) * shape.update_ctas_per_sm;
  return static_cast<unsigned>(ctas < resident ? (ctas ? ctas : 1) : resident);
}

int launch_abs_sum(const float* g, const Geometry& geo, float coef, const Workspace& ws,
                   float* thresholds_out, const LaunchShape& shape, cudaStream_t stream,
                   const unsigned long long* denom) {
  launch_chained(abs_sum_kernel, reduce_grid(geo, shape), kThreads, 0, stream, shape.chained, g, geo, coef, ws,
                 thresholds_out, denom);
  return 1;
}

int launch_abs_max(const float* g, const Geometry& geo, const Workspace& ws,
                   const LaunchShape& shape, cudaStream_t stream) {
  launch_chained(abs_max_kernel, reduce_grid(geo, shape), kThreads, 0, stream, shape.chained, g, geo, ws);
  return 1;
}

int launch_threshold_codes(const float* g, const Geometry& geo, const Workspace& ws,
                           uint32_t* codes, float* scales_out, unsigned long long* counts_out,
                           const LaunchShape& shape, cudaStream_t stream, const uint32_t* indicators) {
  if (indicators)
    launch_chained(threshold_codes_kernel<true>, reduce_grid(geo, shape), kThreads, 0, stream, shape.chained, g, geo, ws,
                   codes, scales_out, counts_out, indicators);
  else
    launch_chained(threshold_codes_kernel<false>, reduce_grid(geo, shape), kThreads, 0, stream, shape.chained, g, geo, ws,
                   codes, scales_out, counts_out, static_cast<const uint32_t*>(nullptr));
  return 1;
}

int launch_stochastic_codes(const float* g, const Geometry& geo, uint64_t seed, uint64_t t,
                            uint32_t stream_base, const Workspace& ws, uint32_t* codes, float* scales_out,
                            unsigned long long* counts_out, const LaunchShape& shape,
                            cudaStream_t stream, const uint32_t* indicators) {
  if (indicators)
    launch_chained(stochastic_codes_kernel<true>, reduce_grid(geo, shape), kThreads, 0, stream, shape.chained, g, geo,
                   philox_key_schedule(seed), t, stream_base, ws, codes, scales_out, counts_out, indicators);
  else
    launch_chained(stochastic_codes_kernel<false>, reduce_grid(geo, shape), kThreads, 0, stream, shape.chained, g, geo,
                   philox_key_schedule(seed), t, stream_base, ws, codes, scales_out, counts_out, static_cast<const uint32_t*>(nullptr));
  return 1;
}

int launch_select_stats(int rule, bool stochastic, const float* g, const Geometry& geo, const float* x,
                        const float* hz, const SelectScalars& sc, float coef, const Workspace& ws,
                        uint32_t* indicators, float* thresholds_out, unsigned long long* selected_out,
                        const LaunchShape& shape, cudaStream_t stream) {
  const size_t smem = select_smem_bytes(geo.M);
  const uint64_t resident = static_cast<uint64_t>(shape.sm_count) * kSelectCtasPerSm;
  const unsigned grid = static_cast<unsigned>(geo.chunks < resident ? geo.chunks : resident);
#define QASG_SELECT(R, S)                                                                                    \
  do {                                                                                                       \
    auto kernel = select_stats_kernel<R, S>;                                                                 \
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(select_smem_bytes(kMaxWorkers))); \
    kernel<<<grid, kThreads, smem, stream>>>(g, geo, x, hz, sc, coef, ws, indicators, thresholds_out, selected_out); \
  } while (0)
  if (rule == 0 && !stochastic) QASG_SELECT(0, false);
  else if (rule == 0) QASG_SELECT(0, true);
  else if (!stochastic) QASG_SELECT(1, false);
  else QASG_SELECT(1, true);
#undef QASG_SELECT
  return 1;
}

int launch_indicator_or(const uint32_t* indicators, uint64_t d, uint32_t M, uint32_t* isyn,
                        unsigned long long* ksyn, const LaunchShape& shape, cudaStream_t stream) {
  const uint64_t words = (d + 31) >> 5;
  const uint64_t ctas = (words + kThreads - 1) / kThreads;
  const uint64_t resident = static_cast<uint64_t>(shape.sm_count) * 8;
  cudaMemsetAsync(ksyn, 0, sizeof(unsigned long long), stream);
  indicator_or_kernel<<<static_cast<unsigned>(ctas < resident ? ctas : resident), kThreads, 0, stream>>>(
      indicators, words, M, isyn, ksyn);
  return 1;
}

// One instantiation of the fused pass C and its launch shape.
template <int kRule, int kM4, int kLanes, int kThreadsC, int kGroups>
static void launch_decode_update_as(const uint32_t* codes, const float* scales, uint64_t d, uint32_t M,
                                    float* x, float* h, float* z, const StepScalars& sc,
                                    unsigned int* status, const LaunchShape& shape, cudaStream_t stream) {
  auto kernel = decode_update_kernel<kRule, kM4, kLanes, kThreadsC, kGroups>;
  const size_t lut_bytes = static_cast<size_t>((M + 3) / 4) * 256 * kLanes * sizeof(double);
  static thread_local int ctas_per_sm[64] = {0};  // per device, resolved on first use
  int dev = 0;
  cudaGetDevice(&dev);
  int& resident = ctas_per_sm[dev & 63];
  if (resident == 0) {
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(lut_bytes));
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kThreadsC, lut_bytes);
    if (resident < 1) resident = 1;
  }
  const uint64_t groups = (d + 3) >> 2;
  const uint64_t per_cta = static_cast<uint64_t>(kThreadsC) * kGroups;
  uint64_t grid = (groups + per_cta - 1) / per_cta;
  const uint64_t max_grid = static_cast<uint64_t>(shape.sm_count) * resident;
  if (grid > max_grid) grid = max_grid;
  const double inv_m = 1.0 / static_cast<double>(M);
  launch_chained(kernel, static_cast<unsigned>(grid), kThreadsC, lut_bytes, stream, shape.chained, codes, scales, d, M,
                 inv_m, x, h, z, sc, status);
}

template <int kRule, int kM4>
static void launch_decode_update_wide_as(const uint32_t* codes, const float* scales, uint64_t d, uint32_t M,
                                         float* x, float* h, float* z, const StepScalars& sc,
                                         unsigned int* status, const LaunchShape& shape, cudaStream_t stream) {
  auto kernel = decode_update_wide_kernel<kRule, kM4>;
  const size_t lut_bytes = static_cast<size_t>(kM4) * kLut3Entries * kLut3Lanes * sizeof(double);
  static thread_local int ctas_per_sm[64] = {0};  // per device, resolved on first use
  int dev = 0;
  cudaGetDevice(&dev);
  int& resident = ctas_per_sm[dev & 63];
  if (resident == 0) {
    cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(lut_bytes));
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kWideThreads, lut_bytes);
    if (resident < 1) resident = 1;
  }
  const uint64_t octs = (d + 7) >> 3;
  uint64_t grid = (octs + kWideThreads - 1) / kWideThreads;
  const uint64_t max_grid = static_cast<uint64_t>(shape.sm_count) * resident;
  if (grid > max_grid) grid = max_grid;
  const double inv_m = 1.0 / static_cast<double>(M);
  launch_chained(kernel, static_cast<unsigned>(grid), kWideThreads, lut_bytes, stream, shape.chained, codes, scales, d, M,
                 inv_m, x, h, z, sc, status);
}

template <int kRule>
static void launch_decode_update_rule(const uint32_t* codes, const float* scales, uint64_t d, uint32_t M,
                                      float* x, float* h, float* z, const StepScalars& sc,
                                      unsigned int* status, const LaunchShape& shape, cudaStream_t stream) {
  constexpr int kG = kRule == 1 ? 1 : 2;  // groups per thread with per-lane tables (measured best)
  // up to 12 workers: 16 copies of the tables (conflict-free for 64-bit lookups), two CTAs of 512 threads per SM
#define QASG_LANES(m4, lanes) \
  case m4: launch_decode_update_as<kRule, m4, lanes, 1024, 1>(codes, scales, d, M, x, h, z, sc, status, shape, stream); break;
#define QASG_WIDE(m4) \
  case m4: \
    if (wide) launch_decode_update_wide_as<kRule, m4>(codes, scales, d, M, x, h, z, sc, status, shape, stream); \
    else launch_decode_update_as<kRule, m4, 8, 1024, 1>(codes, scales, d, M, x, h, z, sc, status, shape, stream); \
    break;
#define QASG_EITHER(m4, prefer_wide) \
  case m4: \
    if constexpr (prefer_wide) { \
      if (wide) { \
        launch_decode_update_wide_as<kRule, m4>(codes, scales, d, M, x, h, z, sc, status, shape, stream); \
        break; \
      } \
    } \
    launch_decode_update_as<kRule, m4, 16, 512, kG>(codes, scales, d, M, x, h, z, sc, status, shape, stream); \
    break;
#define QASG_SHARED(m4) \
  case m4: launch_decode_update_as<kRule, m4, 1, kThreads, 1>(codes, scales, d, M, x, h, z, sc, status, shape, stream); break;
  // the eight-coordinate kernel addresses a worker's code row with a 32-bit byte count
  const bool wide = ((d + 15) >> 4) * 4 <= 0xFFFFFFFFull;
  switch ((M + 3) / 4) {
    // measured at d = 2^28: the eight-coordinate kernel also wins for QCMD from 4 workers on and for QRDA from 9 on
    // (QRDA moves more state per coordinate and loses by loading it after the decode when the decode is short)
    QASG_EITHER(1, kRule == 0) QASG_EITHER(2, kRule == 0) QASG_EITHER(3, kRule != 2)
    QASG_WIDE(4) QASG_WIDE(5) QASG_WIDE(6) QASG_WIDE(7) QASG_WIDE(8)
    // 33 workers and more: 8 copies of the 256-entry tables (two lanes per copy), then one shared copy
    QASG_LANES(9, 8) QASG_LANES(10, 8) QASG_LANES(11, 8) QASG_LANES(12, 8) QASG_LANES(13, 8)
    QASG_SHARED(14) QASG_SHARED(15) QASG_SHARED(16)
  }
#undef QASG_WIDE
#undef QASG_EITHER
#undef QASG_LANES
#undef QASG_SHARED
}

int launch_decode_update(int rule, const uint32_t* codes, const float* scales, uint64_t d,
                         uint32_t M, float* x, float* h, float* z, const StepScalars& sc,
                         unsigned int* status, const LaunchShape& shape, cudaStream_t stream) {
  if (rule == 0)
    launch_decode_update_rule<0>(codes, scales, d, M, x, h, z, sc, status, shape, stream);
  else if (rule == 1)
    launch_decode_update_rule<1>(codes, scales, d, M, x, h, z, sc, status, shape, stream);
  else
    launch_decode_update_rule<2>(codes, scales, d, M, x, h, z, sc, status, shape, stream);
  return 1;
}

template <int kRule, bool kStochastic>
static int launch_fused_step_as(const float* g, const Geometry& geo, const FusedParams& fp, const PhiloxKeys& keys,
                                const Workspace& ws, const Workspace& wsb, StreamSync* sync, uint32_t* codes,
                                float* scales_out, float* x, float* h, float* z, const StepScalars& sc,
                                const LaunchShape& shape, cudaStream_t stream) {
  auto kernel = fused_step_kernel<kRule, kStochastic>;
  const size_t lut_bytes = static_cast<size_t>((geo.M + 3) / 4) * 256 * sizeof(double);
  static thread_local int ctas_per_sm[64] = {0};  // per device, resolved on first use (the table is at most 32 KB)
  int dev = 0;
  cudaGetDevice(&dev);
  int& resident = ctas_per_sm[dev & 63];
  if (resident == 0) {
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&resident, kernel, kThreads, 32768);
    if (resident < 1) resident = 1;
  }
  // enough CTAs for the (worker, chunk) items of passes A and B and for the coordinates of pass C,
  // never more than are resident together
  const uint64_t items = static_cast<uint64_t>(geo.M) * geo.chunks;
  const uint64_t update_ctas = (((geo.d + 3) >> 2) + 2 * kThreads - 1) / (2 * kThreads);
  uint64_t grid = items > update_ctas ? items : update_ctas;
  const uint64_t max_grid = static_cast<uint64_t>(shape.sm_count) * resident;
  if (grid > max_grid) grid = max_grid;
  if (grid < 1) grid = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = lut_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = grid > 1 ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, g, geo, fp, keys, ws, wsb, sync, codes, scales_out, x, h, z, sc);
  return 1;
}

int launch_fused_step(int rule, bool stochastic, const float* g, const Geometry& geo, float coef, uint64_t seed,
                      uint64_t t, uint32_t stream_base, uint32_t max_polls, const Workspace& ws, const Workspace& wsb,
                      StreamSync* sync, uint32_t* codes, float* scales_out, float* x, float* h, float* z,
                      const StepScalars& sc, const LaunchShape& shape, cudaStream_t stream) {
  FusedParams fp;
  fp.coef = coef;
  fp.max_polls = max_polls;
  fp.stream_base = stream_base;
  fp.t = t;
  const PhiloxKeys keys = philox_key_schedule(seed);
  if (rule == 0 && !stochastic)
    return launch_fused_step_as<0, false>(g, geo, fp, keys, ws, wsb, sync, codes, scales_out, x, h, z, sc, shape, stream);
  if (rule == 0)
    return launch_fused_step_as<0, true>(g, geo, fp, keys, ws, wsb, sync, codes, scales_out, x, h, z, sc, shape, stream);
  if (!stochastic)
    return launch_fused_step_as<1, false>(g, geo, fp, keys, ws, wsb, sync, codes, scales_out, x, h, z, sc, shape, stream);
  return launch_fused_step_as<1, true>(g, geo, fp, keys, ws, wsb, sync, codes, scales_out, x, h, z, sc, shape, stream);
}

int launch_decode_average(const uint32_t* codes, const float* scales, uint64_t d, uint32_t M,
                          float* gbar, unsigned int* status, const LaunchShape& shape,
                          cudaStream_t stream) {
  const StepScalars unused = {0.f, 0.f, 0.f, 0.f, 0.f};
  return launch_decode_update(2, codes, scales, d, M, gbar, nullptr, nullptr, unused, status, shape, stream);
}

int launch_dense_update(int rule, const float* q, uint64_t d, float* x, float* h, float* z,
                        const StepScalars& sc, const LaunchShape& shape, cudaStream_t stream) {
  const unsigned grid = update_grid(d, shape);
  if (rule == 0)
    dense_update_kernel<0><<<grid, kThreads, 0, stream>>>(q, d, x, h, z, sc);
  else
    dense_update_kernel<1><<<grid, kThreads, 0, stream>>>(q, d, x, h, z, sc);
  return 1;
}


int launch_mean_update(int rule, const float* g, uint64_t d, uint64_t ld, uint32_t M, float* x, float* h, float* z,
                       const StepScalars& sc, unsigned int* status, const LaunchShape& shape, cudaStream_t stream) {
  const unsigned grid = update_grid(d, shape);
  const double inv_m = 1.0 / static_cast<double>(M);
  if (rule == 0)
    mean_update_kernel<0><<<grid, kThreads, 0, stream>>>(g, d, ld, M, inv_m, x, h, z, sc, status);
  else
    mean_update_kernel<1><<<grid, kThreads, 0, stream>>>(g, d, ld, M, inv_m, x, h, z, sc, status);
  return 1;
}

static unsigned row_grid(const Geometry& geo, const LaunchShape& shape) {
  const uint64_t resident = static_cast<uint64_t>(shape.sm_count) * shape.reduce_ctas_per_sm;
  return static_cast<unsigned>(geo.chunks < resident ? geo.chunks : resident);
}

int launch_avg_stats(bool stochastic, const uint32_t* codes, const float* scales, uint32_t workers,
                     const Geometry& row, float coef, const Workspace& wsq, float* threshold_out,
                     const LaunchShape& shape, cudaStream_t stream, const unsigned long long* denom) {
  const size_t lut_bytes = static_cast<size_t>((workers + 3) / 4) * 256 * sizeof(double);
  const double inv_m = 1.0 / static_cast<double>(workers);
  if (stochastic)
    avg_abs_max_kernel<<<row_grid(row, shape), kThreads, lut_bytes, stream>>>(codes, scales, workers, inv_m, row, wsq);
  else
    avg_abs_sum_kernel<<<row_grid(row, shape), kThreads, lut_bytes, stream>>>(codes, scales, workers, inv_m, row,
                                                                             coef, wsq, threshold_out, denom);
  return 1;
}

int launch_avg_codes(bool stochastic, const uint32_t* codes, const float* scales, uint32_t workers,
                     const Geometry& row, uint64_t seed, uint64_t t, const Workspace& wsq, uint32_t* qcodes,
                     float* scale_out, unsigned long long* count_out, const LaunchShape& shape,
                     cudaStream_t stream) {
  const size_t lut_bytes = static_cast<size_t>((workers + 3) / 4) * 256 * sizeof(double);
  const double inv_m = 1.0 / static_cast<double>(workers);
  if (stochastic)
    avg_codes_kernel<true><<<row_grid(row, shape), kThreads, lut_bytes, stream>>>(
        codes, scales, workers, inv_m, row, seed, t, wsq, qcodes, scale_out, count_out);
  else
    avg_codes_kernel<false><<<row_grid(row, shape), kThreads, lut_bytes, stream>>>(
        codes, scales, workers, inv_m, row, seed, t, wsq, qcodes, scale_out, count_out);
  return 1;
}

}  // namespace qasg

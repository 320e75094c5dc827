// The whole fused step in ONE launch for small dimensions (the dense logistic-regression workload has
// d = 4096): at that size the three kernels of the step are pure launch and latency cost.
//
// CTA m takes worker m's whole row: pass A (sum |g| -> Delta_m) and pass B (codes, s_m) need nothing from
// the other workers, so they run back to back in the same CTA, the second read of the row coming out of
// L1/L2.  The CTA that finishes last then decodes all M code rows and updates x, h (and z).  Every sum is
// taken in the same fixed order as in the large kernels (tile sums, pairwise over tiles), the decode adds
// the workers in the same order, so the results are those of the three-kernel path bit for bit.
#include "qasg_device.cuh"

namespace qasg {

namespace {

template <int kRule>
__global__ void __launch_bounds__(kThreads)
small_step_kernel(const float* __restrict__ g, uint64_t d, uint64_t ld, uint32_t M, uint32_t tiles,
                  uint32_t log2_tiles, float coef, Workspace ws, uint32_t* __restrict__ codes,
                  float* __restrict__ scales_out, float* __restrict__ x, float* __restrict__ h, float* __restrict__ z,
                  StepScalars sc) {
  __shared__ ChunkSumStorage sm_sum;
  __shared__ uint32_t sm_cnt[kThreads / 32];
  __shared__ float sm_delta;
  __shared__ bool sm_last;
  __shared__ float sm_scales[kMaxWorkers];
  const int j = threadIdx.x;
  const uint32_t m = blockIdx.x;
  const float* row = g + static_cast<uint64_t>(m) * ld;
  const uint64_t row_words = (d + 15) >> 4;
  const uint32_t full_tiles = static_cast<uint32_t>(d / kTile);
  ChunkSum chunk_sum(&sm_sum);
  float4 v[kTileRows];

  // pass A: Delta_m = coef * sum|g| / d
  for (uint32_t k = 0; k < tiles; ++k) {
    load_tile(row, static_cast<uint64_t>(k) * kTile, d, j, v);
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
  const double total = chunk_sum.finish(log2_tiles);
  if (j == 0) {
    const float delta = static_cast<float>((static_cast<double>(coef) * total) / static_cast<double>(d));
    sm_delta = delta;
    ws.thresholds[m] = delta;
    if (!isfinite(total)) atomicOr(ws.status, kFlagNonFinite);
  }
  __syncthreads();
  const float delta = sm_delta, ndelta = -delta;

  // pass B: codes and s_m = mean kept magnitude
  uint8_t* codes8 = reinterpret_cast<uint8_t*>(codes + static_cast<uint64_t>(m) * row_words);
  float cntf = 0.f;
  for (uint32_t k = 0; k < tiles; ++k) {
    load_tile(row, static_cast<uint64_t>(k) * kTile, d, j, v);
    double cx = 0.0, cy = 0.0, cz = 0.0, cw = 0.0;
    uint32_t bytes[kTileRows];
#pragma unroll
    for (int r = 0; r < kTileRows; ++r) {
      const float4 t = v[r];
      // strict comparisons; a NaN threshold or value compares false and codes 0
      const float px = t.x > delta ? 1.f : 0.f, nx = t.x < ndelta ? 1.f : 0.f;
      const float py = t.y > delta ? 1.f : 0.f, ny = t.y < ndelta ? 1.f : 0.f;
      const float pz = t.z > delta ? 1.f : 0.f, nz = t.z < ndelta ? 1.f : 0.f;
      const float pw = t.w > delta ? 1.f : 0.f, nw = t.w < ndelta ? 1.f : 0.f;
      const float kx = px + nx, ky = py + ny, kz = pz + nz, kw = pw + nw;
      cx += static_cast<double>(fabsf(t.x) * kx);
      cy += static_cast<double>(fabsf(t.y) * ky);
      cz += static_cast<double>(fabsf(t.z) * kz);
      cw += static_cast<double>(fabsf(t.w) * kw);
      cntf += (kx + ky) + (kz + kw);
      bytes[r] = pack4({px, nx}, {py, ny}, {pz, nz}, {pw, nw});
    }
    store_code_bytes(codes8, k, j, k < full_tiles, row_words * 4, bytes);
    chunk_sum.add_tile((cx + cy) + (cz + cw));
  }
  const double picked = chunk_sum.finish(log2_tiles);
  const unsigned long long n = block_count(static_cast<uint32_t>(cntf), sm_cnt);
  if (j == 0) {
    const float scale = n ? static_cast<float>(picked / static_cast<double>(n)) : 0.f;
    ws.scales[m] = scale;
    ws.counts[m] = n;
    if (scales_out) scales_out[m] = scale;
  }
  __threadfence();  // every thread wrote code bytes: publish them before the CTA takes its ticket
  __syncthreads();
  if (!grid_last_cta(ws.ticket, &sm_last)) return;

  // pass C, by the CTA that finished last: decode, average (Eq. SynQ_t), accumulate, update
  for (uint32_t w = j; w < M; w += kThreads) sm_scales[w] = __ldcg(ws.scales + w);
  __syncthreads();
  const uint8_t* all8 = reinterpret_cast<const uint8_t*>(codes);
  const uint64_t row_bytes = row_words * 4, groups = (d + 3) >> 2;
  const double inv_m = 1.0 / static_cast<double>(M);
  uint32_t bad = 0;
  for (uint64_t grp = j; grp < groups; grp += kThreads) {
    double q[4] = {0.0, 0.0, 0.0, 0.0};
    for (uint32_t g4 = 0; g4 < M; g4 += 4) {  // four workers at a time, as the large kernel's tables do
      double acc[4] = {0.0, 0.0, 0.0, 0.0};
      for (uint32_t w = g4; w < min(g4 + 4, M); ++w) {
        const uint32_t byte = __ldcg(all8 + static_cast<uint64_t>(w) * row_bytes + grp);
        bad |= byte & (byte >> 1) & 0x55u;
        const double sv = static_cast<double>(sm_scales[w]);
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          const uint32_t code = (byte >> (2 * c)) & 3u;
          if (code == 1u) acc[c] += sv;
          else if (code == 2u) acc[c] -= sv;
        }
      }
#pragma unroll
      for (int c = 0; c < 4; ++c) q[c] += acc[c];
    }
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      const uint64_t i = 4 * grp + c;
      if (i >= d) break;
      const float qf = static_cast<float>(q[c] * inv_m);
      float hi = h[i];
      if (kRule == 0) {
        float xi = x[i];
        cmd_update(qf, xi, hi, sc);
        x[i] = xi;
      } else {
        float xi = 0.f, zi = z[i];
        rda_update(qf, xi, hi, zi, sc);
        x[i] = xi;
        z[i] = zi;
      }
      h[i] = hi;
    }
  }
  if (bad) atomicOr(ws.status, kFlagBadCode);
  if (j == 0) *ws.ticket = 0u;
}

}  // namespace

int launch_small_step(int rule, const float* g, uint64_t d, uint64_t ld, uint32_t M, float coef, const Workspace& ws,
                      uint32_t* codes, float* scales_out, float* x, float* h, float* z, const StepScalars& sc,
                      cudaStream_t stream) {
  const uint32_t tiles = static_cast<uint32_t>((d + kTile - 1) / kTile);
  uint32_t log2_tiles = 0;
  while ((1u << log2_tiles) < tiles) ++log2_tiles;
  if (rule == 0)
    small_step_kernel<0><<<M, kThreads, 0, stream>>>(g, d, ld, M, tiles, log2_tiles, coef, ws, codes, scales_out, x, h, z, sc);
  else
    small_step_kernel<1><<<M, kThreads, 0, stream>>>(g, d, ld, M, tiles, log2_tiles, coef, ws, codes, scales_out, x, h, z, sc);
  return 1;
}

}  // namespace qasg

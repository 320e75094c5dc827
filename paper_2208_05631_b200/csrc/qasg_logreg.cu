// Per-worker minibatch gradient of logistic regression (the linear-model workload):
//   g_m = (1/B) sum_j -y_j * sigmoid(-y_j <a_j, x>) * a_j
// Dense: GEMV-shaped and memory-bound.  Kernel 1 computes one coefficient per minibatch
// row (a warp per row, 128-bit loads); kernel 2 forms the coefficient-weighted column sums
// with a fixed summation order, reading the rows a second time out of L2.
// CSR: one warp per minibatch row computes the margin and scatters with atomic adds.  The sparse form
// keeps the dense rows of g zero between calls and a bit per entry that a minibatch touched, so a call
// moves the touched sectors only (no clearing or re-reading of M*d floats).
#include "qasg_device.cuh"

namespace qasg {

struct Shards {
  uint64_t row0[kMaxWorkers + 1];
};

// Global row id of minibatch entry b of worker m.
__device__ __forceinline__ uint64_t batch_row(const Shards& sh, const uint32_t* __restrict__ batch_rows,
                                              uint32_t m, uint32_t b, uint32_t B, uint64_t t) {
  if (batch_rows) return batch_rows[static_cast<uint64_t>(m) * B + b];
  const uint64_t lo = sh.row0[m], n = sh.row0[m + 1] - lo;
  return lo + ((t - 1) % n * (B % n) + b) % n;
}

// -y * sigmoid(-y * s) / B, evaluated without overflow.
__device__ __forceinline__ float logistic_coef(float y, float s, float inv_b) {
  const float v = -y * s;
  float sig;
  if (v >= 0.f) {
    sig = 1.f / (1.f + expf(-v));
  } else {
    const float e = expf(v);
    sig = e / (1.f + e);
  }
  return -y * sig * inv_b;
}

__global__ void __launch_bounds__(kThreads)
logreg_dense_coef_kernel(const float* __restrict__ X, const float* __restrict__ y, uint64_t n_rows, uint64_t d,
                         uint32_t M, Shards sh, const uint32_t* __restrict__ batch_rows, uint32_t B, uint64_t t,
                         const float* __restrict__ x, float* __restrict__ coef, uint32_t* __restrict__ rows,
                         unsigned int* __restrict__ status) {
  const uint32_t warp = (blockIdx.x * kThreads + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  chain_wait();  // x comes from the update of the iteration before
  chain_trigger();
  if (warp >= M * B) return;
  const uint32_t m = warp / B, b = warp - m * B;
  const uint64_t r = batch_row(sh, batch_rows, m, b, B, t);
  if (r >= n_rows) {  // a caller's row id outside the matrix: the row adds nothing
    if (lane == 0) {
      coef[warp] = 0.f;
      rows[warp] = 0u;
      atomicOr(status, kFlagBadIndex);
    }
    return;
  }
  const float4* a = reinterpret_cast<const float4*>(X + r * d);
  const float4* xv = reinterpret_cast<const float4*>(x);
  float acc = 0.f;
  for (uint64_t k = lane; k < (d >> 2); k += 32) {
    const float4 u = __ldg(a + k), w = __ldg(xv + k);
    acc = fmaf(u.x, w.x, acc);
    acc = fmaf(u.y, w.y, acc);
    acc = fmaf(u.z, w.z, acc);
    acc = fmaf(u.w, w.w, acc);
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
  if (lane == 0) {
    coef[warp] = logistic_coef(y[r], acc, 1.f / static_cast<float>(B));
    rows[warp] = static_cast<uint32_t>(r);
  }
}

// grid (d/128, M), 1024 threads: thread (cq = tid & 31 -> 4 columns, rl = tid >> 5 -> rows rl, rl+32, ...).
// The 32 row lanes are combined in lane order, so the result does not depend on timing.
constexpr int kColsumThreads = 1024;
__global__ void __launch_bounds__(kColsumThreads)
logreg_dense_colsum_kernel(const float* __restrict__ X, uint64_t d, uint32_t B, const float* __restrict__ coef,
                           const uint32_t* __restrict__ rows, float* __restrict__ g, uint64_t ld_g) {
  constexpr int kRowLanes = kColsumThreads / 32;
  __shared__ float4 sm[kRowLanes][32];
  chain_wait();  // the coefficients come from the launch before this one
  chain_trigger();
  const uint32_t m = blockIdx.y, cq = threadIdx.x & 31, rl = threadIdx.x >> 5;
  const uint64_t col = (static_cast<uint64_t>(blockIdx.x) * 32 + cq) * 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  if (col < d) {
    const float* cm = coef + static_cast<uint64_t>(m) * B;
    const uint32_t* rm = rows + static_cast<uint64_t>(m) * B;
#pragma unroll 4
    for (uint32_t b = rl; b < B; b += kRowLanes) {
      const float c = cm[b];
      const float4 a = __ldg(reinterpret_cast<const float4*>(X + static_cast<uint64_t>(rm[b]) * d + col));
      acc.x = fmaf(c, a.x, acc.x);
      acc.y = fmaf(c, a.y, acc.y);
      acc.z = fmaf(c, a.z, acc.z);
      acc.w = fmaf(c, a.w, acc.w);
    }
  }
  sm[rl][cq] = acc;
  __syncthreads();
  if (rl == 0 && col < d) {
#pragma unroll
    for (int k = 1; k < kRowLanes; ++k) {
      const float4 o = sm[k][cq];
      acc.x += o.x;
      acc.y += o.y;
      acc.z += o.z;
      acc.w += o.w;
    }
    *reinterpret_cast<float4*>(g + static_cast<uint64_t>(m) * ld_g + col) = acc;
  }
}

// grid (ceil(B / 8), M): a CTA takes 8 minibatch rows of one worker, a warp per row.  Columns below
// kHotCols are accumulated in shared memory first and reach g with one atomic per CTA and column:
// with Zipf-like column frequencies nearly every row holds the first few columns, and same-address
// atomics in L2 serialise.
constexpr uint32_t kHotCols = 4096;
template <bool kTouched>
__global__ void __launch_bounds__(kThreads)
logreg_csr_kernel(const int64_t* __restrict__ rowptr, const int32_t* __restrict__ colidx,
                  const float* __restrict__ vals, const float* __restrict__ y, uint64_t n_rows, uint64_t d,
                  Shards sh, const uint32_t* __restrict__ batch_rows, uint32_t B, uint64_t t,
                  const float* __restrict__ x, float* __restrict__ g, uint64_t ld_g, uint32_t* __restrict__ touched,
                  uint64_t touched_words, unsigned int* __restrict__ status) {
  __shared__ float hot[kHotCols];
  __shared__ uint32_t hot_bits[kHotCols / 32];
  const uint32_t m = blockIdx.y, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t b = blockIdx.x * (kThreads / 32) + warp;
  for (uint32_t c = threadIdx.x; c < kHotCols; c += kThreads) hot[c] = 0.f;
  if (threadIdx.x < kHotCols / 32) hot_bits[threadIdx.x] = 0u;
  __syncthreads();
  float* row = g + static_cast<uint64_t>(m) * ld_g;
  // Indices come from the caller's data: a row id, a rowptr pair or a column outside its range is
  // skipped and reported, never used as an address.
  bool bad_index = false;
  const uint64_t r = b < B ? batch_row(sh, batch_rows, m, b, B, t) : 0;
  int64_t lo = 0, hi = 0;
  if (b < B) {
    if (r < n_rows) {
      lo = rowptr[r];
      hi = rowptr[r + 1];
      if (lo < 0 || hi < lo || hi > rowptr[n_rows]) {
        bad_index = true;
        hi = lo = 0;
      }
    } else {
      bad_index = true;
    }
  }
  if (b < B && hi > lo) {
    float acc = 0.f;
    for (int64_t k = lo + lane; k < hi; k += 32) {
      const int32_t col = __ldg(colidx + k);
      if (col >= 0 && static_cast<uint64_t>(col) < d) acc = fmaf(__ldg(vals + k), __ldg(x + col), acc);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, s);
    const float c = logistic_coef(y[r], acc, 1.f / static_cast<float>(B));
    uint32_t* bits = kTouched ? touched + static_cast<uint64_t>(m) * touched_words : nullptr;
    for (int64_t k = lo + lane; k < hi; k += 32) {
      const int32_t signed_col = __ldg(colidx + k);
      if (signed_col < 0 || static_cast<uint64_t>(signed_col) >= d) {
        bad_index = true;
        continue;
      }
      const uint32_t col = static_cast<uint32_t>(signed_col);
      const float add = c * __ldg(vals + k);
      const uint32_t bit = 1u << (col & 31u);
      if (col < kHotCols) {
        atomicAdd(hot + col, add);
        if (kTouched) atomicOr(hot_bits + (col >> 5), bit);
      } else {
        atomicAdd(row + col, add);
        // look before the atomic: a set bit needs no second write
        if (kTouched && !(__ldcg(bits + (col >> 5)) & bit)) atomicOr(bits + (col >> 5), bit);
      }
    }
  }
  if (bad_index) atomicOr(status, kFlagBadIndex);
  __syncthreads();
  const uint32_t hot_cols = d < kHotCols ? static_cast<uint32_t>(d) : kHotCols;
  for (uint32_t c = threadIdx.x; c < hot_cols; c += kThreads) {
    const float v = hot[c];
    if (v != 0.f) atomicAdd(row + c, v);
  }
  if (kTouched && threadIdx.x < kHotCols / 32 && threadIdx.x < touched_words) {
    uint32_t* word = touched + static_cast<uint64_t>(m) * touched_words + threadIdx.x;
    const uint32_t mine = hot_bits[threadIdx.x];
    if (mine & ~__ldcg(word)) atomicOr(word, mine);
  }
}

// Zeroes the entries of g the bits mark, then the bits.  The M rows of bits are one flat array; a
// thread takes four words at a time (one 128-bit load; nearly all of them are zero).
__device__ __forceinline__ void clear_marked(float* __restrict__ g, uint64_t ld_g, uint64_t touched_words, uint64_t d,
                                             uint64_t w, uint32_t bits) {
  const uint64_t m = w / touched_words, word = w - m * touched_words;
  float* base = g + m * ld_g + word * 32;
  while (bits) {
    const int b = __ffs(bits) - 1;
    if (word * 32 + b < d) base[b] = 0.f;  // a stray bit past d marks nothing
    bits &= bits - 1;
  }
}

__global__ void __launch_bounds__(kThreads)
touched_clear_kernel(float* __restrict__ g, uint64_t ld_g, uint32_t M, uint32_t* __restrict__ touched,
                     uint64_t touched_words, uint64_t d) {
  const uint64_t total = static_cast<uint64_t>(M) * touched_words, quads = total >> 2;
  const uint64_t tid = static_cast<uint64_t>(blockIdx.x) * kThreads + threadIdx.x;
  const uint64_t stride = static_cast<uint64_t>(gridDim.x) * kThreads;
  uint4* t4 = reinterpret_cast<uint4*>(touched);
  for (uint64_t q = tid; q < quads; q += stride) {
    const uint4 v = t4[q];
    if (!(v.x | v.y | v.z | v.w)) continue;
    if (v.x) clear_marked(g, ld_g, touched_words, d, 4 * q, v.x);
    if (v.y) clear_marked(g, ld_g, touched_words, d, 4 * q + 1, v.y);
    if (v.z) clear_marked(g, ld_g, touched_words, d, 4 * q + 2, v.z);
    if (v.w) clear_marked(g, ld_g, touched_words, d, 4 * q + 3, v.w);
    t4[q] = make_uint4(0u, 0u, 0u, 0u);
  }
  for (uint64_t w = 4 * quads + tid; w < total; w += stride) {
    const uint32_t bits = touched[w];
    if (bits) {
      clear_marked(g, ld_g, touched_words, d, w, bits);
      touched[w] = 0u;
    }
  }
}

static Shards make_shards(const uint64_t* shard_row0_host, uint32_t M) {
  Shards sh;
  for (uint32_t m = 0; m <= M; ++m) sh.row0[m] = shard_row0_host[m];
  return sh;
}

int launch_logreg_dense(const float* X, const float* y, uint64_t n_rows, uint64_t d, uint32_t M,
                        const uint64_t* shard_row0_host, const uint32_t* batch_rows, uint32_t B,
                        uint64_t t, const float* x, float* g, uint64_t ld_g, float* coef_ws,
                        unsigned int* status, const LaunchShape& shape, cudaStream_t stream) {
  const Shards sh = make_shards(shard_row0_host, M);
  uint32_t* rows_ws = reinterpret_cast<uint32_t*>(coef_ws + static_cast<uint64_t>(M) * B);
  const uint64_t warps = static_cast<uint64_t>(M) * B;
  const unsigned grid1 = static_cast<unsigned>((warps * 32 + kThreads - 1) / kThreads);
  launch_chained(logreg_dense_coef_kernel, grid1, kThreads, 0, stream, shape.chained, X, y, n_rows, d, M, sh, batch_rows, B,
                 t, x, coef_ws, rows_ws, status);
  cudaLaunchConfig_t cfg = {};  // a two-dimensional grid: (column blocks, workers)
  cfg.gridDim = dim3(static_cast<unsigned>((d + 127) / 128), M);
  cfg.blockDim = dim3(kColsumThreads);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = shape.chained ? 1 : 0;
  cudaLaunchKernelEx(&cfg, logreg_dense_colsum_kernel, X, d, B, static_cast<const float*>(coef_ws),
                     static_cast<const uint32_t*>(rows_ws), g, ld_g);
  return 2;
}

int launch_logreg_csr(const int64_t* rowptr, const int32_t* colidx, const float* vals,
                      const float* y, uint64_t n_rows, uint64_t d, uint32_t M, const uint64_t* shard_row0_host,
                      const uint32_t* batch_rows, uint32_t B, uint64_t t, const float* x, float* g,
                      uint64_t ld_g, unsigned int* status, const LaunchShape&, cudaStream_t stream,
                      uint32_t* touched) {
  const Shards sh = make_shards(shard_row0_host, M);
  const dim3 grid((B + kThreads / 32 - 1) / (kThreads / 32), M);
  if (touched) {
    logreg_csr_kernel<true><<<grid, kThreads, 0, stream>>>(rowptr, colidx, vals, y, n_rows, d, sh, batch_rows, B, t, x,
                                                          g, ld_g, touched, (d + 31) >> 5, status);
  } else {
    cudaMemset2DAsync(g, ld_g * sizeof(float), 0, d * sizeof(float), M, stream);
    logreg_csr_kernel<false><<<grid, kThreads, 0, stream>>>(rowptr, colidx, vals, y, n_rows, d, sh, batch_rows, B, t, x,
                                                           g, ld_g, nullptr, 0, status);
  }
  return 1;
}

int launch_touched_clear(float* g, uint64_t d, uint64_t ld_g, uint32_t M, uint32_t* touched,
                         const LaunchShape& shape, cudaStream_t stream) {
  const uint64_t words = (d + 31) >> 5;
  const uint64_t ctas = (static_cast<uint64_t>(M) * words / 4 + kThreads) / kThreads;
  const uint64_t cap = static_cast<uint64_t>(shape.sm_count) * 8;
  touched_clear_kernel<<<static_cast<unsigned>(ctas < cap ? ctas : cap), kThreads, 0, stream>>>(g, ld_g, M, touched,
                                                                                              words, d);
  return 1;
}

}  // namespace qasg

// Exact optimal threshold of the threshold quantizer (Section 3.4): rank the magnitudes of a worker's
// gradient, take every component as a candidate threshold, keep the one that maximises
//   F_k = (sum of the k largest |v|)^2 / k .
// The paper replaces this O(d log d) procedure by the 0.75 * mean|v| rule; it is built here so that the
// rule can be checked against it at full size.
//
//   sort      least-significant-digit radix sort of the magnitudes' bit patterns (descending |v|):
//             8 passes of 4 bits; per pass a per-tile histogram, a scan of the (digit, tile) counts and
//             a stable scatter (a thread owns 16 consecutive keys and private counters, so ranks follow
//             the input order without atomics)
//   prefix    fixed-order fp64 prefix sums of the ranked magnitudes: blocks of 1024 (doubling scan
//             in each warp, doubling scan of the 32 warp totals), groups of 1024 blocks scanned the
//             same way, groups added one after the other
//   pick      F_k at every strict drop of the ranked magnitudes, first maximum, Delta* = the largest
//             component outside the chosen set
#include "qasg_internal.h"

namespace qasg {

namespace {

constexpr int kSortThreads = 256;
constexpr int kKeysPerThread = 16;
constexpr int kSortTile = kSortThreads * kKeysPerThread;  // 4096 keys per CTA
constexpr int kRadixBits = 4;
constexpr int kRadix = 1 << kRadixBits;
constexpr int kSortPasses = 8;         // 31 significant key bits
constexpr int kScanChunk = 4096;       // (digit, tile) counts scanned per CTA
constexpr int kBlock = 1024;           // prefix-sum block, one element per thread

// Ascending keys rank descending magnitudes (bit patterns of non-negative floats order like their values).
__device__ __forceinline__ uint32_t magnitude_key(uint32_t bits) { return 0x7FFFFFFFu - (bits & 0x7FFFFFFFu); }
__device__ __forceinline__ float key_magnitude(uint32_t key) { return __uint_as_float(0x7FFFFFFFu - key); }

// The 16 consecutive keys thread tid owns in tile `tile`; `valid` of them lie below n.
template <bool kFromFloat>
__device__ __forceinline__ void load_thread_keys(const uint32_t* __restrict__ src, uint64_t n, uint32_t tile,
                                                 uint32_t (&key)[kKeysPerThread], int& valid) {
  const uint64_t base = static_cast<uint64_t>(tile) * kSortTile + threadIdx.x * kKeysPerThread;
  valid = base >= n ? 0 : (n - base >= kKeysPerThread ? kKeysPerThread : static_cast<int>(n - base));
  if (valid == kKeysPerThread) {
    const uint4* p = reinterpret_cast<const uint4*>(src + base);
#pragma unroll
    for (int q = 0; q < kKeysPerThread / 4; ++q) {
      const uint4 v = __ldg(p + q);
      key[4 * q] = v.x, key[4 * q + 1] = v.y, key[4 * q + 2] = v.z, key[4 * q + 3] = v.w;
    }
  } else {
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) key[e] = e < valid ? __ldg(src + base + e) : 0u;
  }
  if (kFromFloat) {
#pragma unroll
    for (int e = 0; e < kKeysPerThread; ++e) key[e] = magnitude_key(key[e]);
  }
}

// counts[digit * ntiles + tile] = keys of the tile with that digit.
template <bool kFromFloat>
__global__ void __launch_bounds__(kSortThreads)
sort_hist_kernel(const uint32_t* __restrict__ src, uint64_t n, uint32_t shift, uint32_t ntiles,
                 uint32_t* __restrict__ counts, unsigned int* __restrict__ status) {
  __shared__ uint32_t hist[kSortThreads / 32][kRadix];
  const uint32_t tile = blockIdx.x, warp = threadIdx.x >> 5;
  if (threadIdx.x < (kSortThreads / 32) * kRadix) (&hist[0][0])[threadIdx.x] = 0u;
  __syncthreads();
  uint32_t key[kKeysPerThread];
  int valid;
  load_thread_keys<kFromFloat>(src, n, tile, key, valid);
  bool nonfinite = false;
#pragma unroll
  for (int e = 0; e < kKeysPerThread; ++e)
    if (e < valid) {
      atomicAdd(&hist[warp][(key[e] >> shift) & (kRadix - 1)], 1u);
      if (kFromFloat) nonfinite |= key[e] <= 0x007FFFFFu;  // |v| is Inf or NaN
    }
  if (kFromFloat && nonfinite) atomicOr(status, kFlagNonFinite);
  __syncthreads();
  if (threadIdx.x < kRadix) {
    uint32_t total = 0;
#pragma unroll
    for (int w = 0; w < kSortThreads / 32; ++w) total += hist[w][threadIdx.x];
    counts[static_cast<uint64_t>(threadIdx.x) * ntiles + tile] = total;
  }
}

// Exclusive prefix of one value per thread over a CTA of kSortThreads threads; `total` gets the CTA sum.
__device__ __forceinline__ uint32_t block_exclusive_scan(uint32_t v, uint32_t* sm_warp, uint32_t& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t incl = v;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const uint32_t y = __shfl_up_sync(0xffffffffu, incl, s);
    if (lane >= s) incl += y;
  }
  __syncthreads();  // sm_warp may still be read from a previous call
  if (lane == 31) sm_warp[warp] = incl;
  __syncthreads();
  uint32_t before = 0;
  total = 0;
#pragma unroll
  for (int w = 0; w < kSortThreads / 32; ++w) {
    if (w < warp) before += sm_warp[w];
    total += sm_warp[w];
  }
  return before + incl - v;
}

// Exclusive scan of the counts inside chunks of kScanChunk entries; chunk totals to chunk_total.
// len is a multiple of 16 (16 digits times the number of tiles).
__global__ void __launch_bounds__(kSortThreads)
sort_scan_chunks_kernel(uint32_t* __restrict__ counts, uint64_t len, uint32_t* __restrict__ chunk_total) {
  __shared__ uint32_t sm_warp[kSortThreads / 32];
  const uint64_t base = static_cast<uint64_t>(blockIdx.x) * kScanChunk + threadIdx.x * 16;
  uint32_t v[16];
  uint32_t run = 0;
  if (base < len) {
    const uint4* p = reinterpret_cast<const uint4*>(counts + base);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint4 t = p[q];
      v[4 * q] = t.x, v[4 * q + 1] = t.y, v[4 * q + 2] = t.z, v[4 * q + 3] = t.w;
    }
#pragma unroll
    for (int e = 0; e < 16; ++e) {
      const uint32_t t = v[e];
      v[e] = run;
      run += t;
    }
  }
  uint32_t total;
  const uint32_t before = block_exclusive_scan(run, sm_warp, total);
  if (base < len) {
    uint4* p = reinterpret_cast<uint4*>(counts + base);
#pragma unroll
    for (int q = 0; q < 4; ++q)
      p[q] = make_uint4(before + v[4 * q], before + v[4 * q + 1], before + v[4 * q + 2], before + v[4 * q + 3]);
  }
  if (threadIdx.x == 0) chunk_total[blockIdx.x] = total;
}

// Exclusive scan, in place, of the chunk totals (one CTA; a running carry across rounds of 256).
__global__ void __launch_bounds__(kSortThreads)
sort_scan_totals_kernel(uint32_t* __restrict__ chunk_total, uint32_t nchunks) {
  __shared__ uint32_t sm_warp[kSortThreads / 32];
  uint32_t carry = 0;
  for (uint32_t base = 0; base < nchunks; base += kSortThreads) {
    const uint32_t i = base + threadIdx.x;
    const uint32_t v = i < nchunks ? chunk_total[i] : 0u;
    uint32_t total;
    const uint32_t before = block_exclusive_scan(v, sm_warp, total);
    if (i < nchunks) chunk_total[i] = carry + before;
    carry += total;
  }
}

// Stable scatter of one digit.  A thread's 16 keys are consecutive in the input, its counters are
// private (cnt[digit][thread]); scanning the counters digit-major, thread-minor gives every thread the
// tile-local rank of its first key of each digit, and ranks then follow the input order.  The tile is
// reordered in shared memory and leaves in runs of equal digit.
template <bool kFromFloat>
__global__ void __launch_bounds__(kSortThreads)
sort_scatter_kernel(const uint32_t* __restrict__ src, uint32_t* __restrict__ dst, uint64_t n, uint32_t shift,
                    uint32_t ntiles, const uint32_t* __restrict__ counts, const uint32_t* __restrict__ chunk_before) {
  __shared__ uint16_t cnt[kRadix][kSortThreads];
  __shared__ uint32_t keys_sm[kSortTile];
  __shared__ uint32_t sm_warp[kSortThreads / 32];
  __shared__ uint32_t digit_start[kRadix], digit_dst[kRadix];
  const uint32_t tile = blockIdx.x, tid = threadIdx.x;
  uint32_t key[kKeysPerThread];
  int valid;
  load_thread_keys<kFromFloat>(src, n, tile, key, valid);
#pragma unroll
  for (int dg = 0; dg < kRadix; ++dg) cnt[dg][tid] = 0;
#pragma unroll
  for (int e = 0; e < kKeysPerThread; ++e)
    if (e < valid) ++cnt[(key[e] >> shift) & (kRadix - 1)][tid];
  if (tid < kRadix) {
    const uint64_t idx = static_cast<uint64_t>(tid) * ntiles + tile;
    digit_dst[tid] = counts[idx] + chunk_before[idx / kScanChunk];
  }
  __syncthreads();
  // linear order digit * 256 + thread: thread tid scans entries 16*tid .. 16*tid + 15 (digit tid >> 4)
  uint16_t* lin = &cnt[0][0];
  uint32_t local[16], run = 0;
#pragma unroll
  for (int e = 0; e < 16; ++e) {
    local[e] = run;
    run += lin[16 * tid + e];
  }
  uint32_t total;
  const uint32_t before = block_exclusive_scan(run, sm_warp, total);
#pragma unroll
  for (int e = 0; e < 16; ++e) lin[16 * tid + e] = static_cast<uint16_t>(before + local[e]);
  if ((tid & 15u) == 0) digit_start[tid >> 4] = before;  // rank of the digit's first key in the tile
  __syncthreads();
#pragma unroll
  for (int e = 0; e < kKeysPerThread; ++e)
    if (e < valid) {
      const uint32_t dg = (key[e] >> shift) & (kRadix - 1);
      keys_sm[cnt[dg][tid]++] = key[e];
    }
  __syncthreads();
  const uint64_t tile_base = static_cast<uint64_t>(tile) * kSortTile;
  const uint32_t tile_n = n - tile_base >= kSortTile ? kSortTile : static_cast<uint32_t>(n - tile_base);
  for (uint32_t i = tid; i < tile_n; i += kSortThreads) {
    const uint32_t k = keys_sm[i];
    const uint32_t dg = (k >> shift) & (kRadix - 1);
    dst[digit_dst[dg] + (i - digit_start[dg])] = k;
  }
}

// Inclusive fp64 scan of one value per thread over a CTA of 1024 threads in the fixed order:
// doubling scan in each warp, doubling scan of the 32 warp totals, (warps before) + (value in the warp).
__device__ __forceinline__ double block_scan_1024(double x, double* sm_warp) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int s = 1; s < 32; s <<= 1) {
    const double y = __shfl_up_sync(0xffffffffu, x, s);
    if (lane >= s) x = __dadd_rn(y, x);
  }
  __syncthreads();
  if (lane == 31) sm_warp[warp] = x;
  __syncthreads();
  if (warp == 0) {
    double t = sm_warp[lane];
#pragma unroll
    for (int s = 1; s < 32; s <<= 1) {
      const double y = __shfl_up_sync(0xffffffffu, t, s);
      if (lane >= s) t = __dadd_rn(y, t);
    }
    sm_warp[32 + lane] = t;
  }
  __syncthreads();
  const double before = warp ? sm_warp[32 + warp - 1] : 0.0;
  return __dadd_rn(before, x);
}

// Totals of the blocks of 1024 ranked magnitudes.
__global__ void __launch_bounds__(kBlock)
prefix_block_totals_kernel(const uint32_t* __restrict__ keys, uint64_t n, double* __restrict__ block_total) {
  __shared__ double sm_warp[64];
  const uint64_t i = static_cast<uint64_t>(blockIdx.x) * kBlock + threadIdx.x;
  const double x = i < n ? static_cast<double>(key_magnitude(__ldg(keys + i))) : 0.0;
  const double incl = block_scan_1024(x, sm_warp);
  if (threadIdx.x == kBlock - 1) block_total[blockIdx.x] = incl;
}

// One CTA per group of 1024 blocks: inclusive scan of the block totals inside the group.
__global__ void __launch_bounds__(kBlock)
prefix_group_scan_kernel(const double* __restrict__ block_total, uint32_t nblocks, double* __restrict__ block_incl,
                         double* __restrict__ group_total) {
  __shared__ double sm_warp[64];
  const uint32_t b = blockIdx.x * kBlock + threadIdx.x;
  const double incl = block_scan_1024(b < nblocks ? block_total[b] : 0.0, sm_warp);
  if (b < nblocks) block_incl[b] = incl;
  if (threadIdx.x == kBlock - 1) group_total[blockIdx.x] = incl;
}

// groups_before[g] = total of the groups before g, added one after the other (one thread).
__global__ void prefix_groups_kernel(const double* __restrict__ group_total, uint32_t ngroups,
                                     double* __restrict__ groups_before) {
  if (threadIdx.x || blockIdx.x) return;
  double acc = 0.0;
  for (uint32_t g = 0; g < ngroups; ++g) {
    groups_before[g] = acc;
    acc = __dadd_rn(acc, group_total[g]);
  }
}

struct Candidate {
  double f;    // objective, -1 when the block holds no candidate
  uint32_t i;  // rank (0-based) of the last kept magnitude
};
__device__ __forceinline__ bool better(double f, uint32_t i, double g, uint32_t j) {
  return f > g || (f == g && i < j);
}

// Objective at every strict drop of the ranked magnitudes of one block; the block's first maximum.
__global__ void __launch_bounds__(kBlock)
objective_kernel(const uint32_t* __restrict__ keys, uint64_t n, const double* __restrict__ block_incl,
                 const double* __restrict__ groups_before, double* __restrict__ cand_f,
                 uint32_t* __restrict__ cand_i) {
  __shared__ double sm_warp[64];
  __shared__ double sm_f[32];
  __shared__ uint32_t sm_i[32];
  const uint32_t b = blockIdx.x;
  const uint64_t i = static_cast<uint64_t>(b) * kBlock + threadIdx.x;
  const float a = i < n ? key_magnitude(__ldg(keys + i)) : 0.f;
  const double inside = block_scan_1024(static_cast<double>(a), sm_warp);
  const double blocks_before = (b % kBlock) ? block_incl[b - 1] : 0.0;
  const double prefix = __dadd_rn(__dadd_rn(groups_before[b / kBlock], blocks_before), inside);
  double f = -1.0;
  if (i < n && a > 0.f) {
    const bool drop = i + 1 == n || key_magnitude(__ldg(keys + i + 1)) < a;
    if (drop) f = __ddiv_rn(__dmul_rn(prefix, prefix), static_cast<double>(i + 1));
  }
  uint32_t idx = static_cast<uint32_t>(i);
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    const double of = __shfl_xor_sync(0xffffffffu, f, s);
    const uint32_t oi = __shfl_xor_sync(0xffffffffu, idx, s);
    if (better(of, oi, f, idx)) f = of, idx = oi;
  }
  if ((threadIdx.x & 31) == 0) sm_f[threadIdx.x >> 5] = f, sm_i[threadIdx.x >> 5] = idx;
  __syncthreads();
  if (threadIdx.x < 32) {
    f = sm_f[threadIdx.x], idx = sm_i[threadIdx.x];
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
      const double of = __shfl_xor_sync(0xffffffffu, f, s);
      const uint32_t oi = __shfl_xor_sync(0xffffffffu, idx, s);
      if (better(of, oi, f, idx)) f = of, idx = oi;
    }
    if (threadIdx.x == 0) cand_f[b] = f, cand_i[b] = idx;
  }
}

// One CTA: the first maximum over all blocks; Delta* = the largest magnitude outside the chosen set.
__global__ void __launch_bounds__(kBlock)
pick_kernel(const uint32_t* __restrict__ keys, uint64_t n, const double* __restrict__ cand_f,
            const uint32_t* __restrict__ cand_i, uint32_t nblocks, float* __restrict__ ws_threshold,
            float* __restrict__ threshold_out, unsigned long long* __restrict__ kept_out) {
  __shared__ double sm_f[32];
  __shared__ uint32_t sm_i[32];
  double f = -1.0;
  uint32_t idx = 0xffffffffu;
  for (uint32_t b = threadIdx.x; b < nblocks; b += kBlock) {
    const double of = cand_f[b];
    const uint32_t oi = cand_i[b];
    if (better(of, oi, f, idx)) f = of, idx = oi;
  }
#pragma unroll
  for (int s = 16; s > 0; s >>= 1) {
    const double of = __shfl_xor_sync(0xffffffffu, f, s);
    const uint32_t oi = __shfl_xor_sync(0xffffffffu, idx, s);
    if (better(of, oi, f, idx)) f = of, idx = oi;
  }
  if ((threadIdx.x & 31) == 0) sm_f[threadIdx.x >> 5] = f, sm_i[threadIdx.x >> 5] = idx;
  __syncthreads();
  if (threadIdx.x < 32) {
    f = sm_f[threadIdx.x], idx = sm_i[threadIdx.x];
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
      const double of = __shfl_xor_sync(0xffffffffu, f, s);
      const uint32_t oi = __shfl_xor_sync(0xffffffffu, idx, s);
      if (better(of, oi, f, idx)) f = of, idx = oi;
    }
    if (threadIdx.x == 0) {
      float delta = 0.f;
      unsigned long long kept = 0;
      if (f >= 0.0) {
        kept = static_cast<unsigned long long>(idx) + 1;
        if (kept < n) delta = key_magnitude(keys[kept]);
      }
      *ws_threshold = delta;
      if (threshold_out) *threshold_out = delta;
      if (kept_out) *kept_out = kept;
    }
  }
}

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

struct OptimalScratch {
  uint32_t *keys_a, *keys_b, *counts, *chunk_total, *cand_i;
  double *block_total, *block_incl, *group_total, *groups_before, *cand_f;
  uint64_t bytes;
};

OptimalScratch carve(void* base, uint64_t d) {
  const uint64_t ntiles = (d + kSortTile - 1) / kSortTile, nblocks = (d + kBlock - 1) / kBlock;
  const uint64_t nchunks = (kRadix * ntiles + kScanChunk - 1) / kScanChunk, ngroups = (nblocks + kBlock - 1) / kBlock;
  uint64_t off = 0;
  auto take = [&](uint64_t bytes) {
    const uint64_t at = off;
    off = align_up(off + bytes, 256);
    return reinterpret_cast<char*>(base) + at;
  };
  OptimalScratch s;
  s.keys_a = reinterpret_cast<uint32_t*>(take(ntiles * kSortTile * 4));
  s.keys_b = reinterpret_cast<uint32_t*>(take(ntiles * kSortTile * 4));
  s.counts = reinterpret_cast<uint32_t*>(take(kRadix * ntiles * 4));
  s.chunk_total = reinterpret_cast<uint32_t*>(take(nchunks * 4));
  s.cand_i = reinterpret_cast<uint32_t*>(take(nblocks * 4));
  s.block_total = reinterpret_cast<double*>(take(nblocks * 8));
  s.block_incl = reinterpret_cast<double*>(take(nblocks * 8));
  s.group_total = reinterpret_cast<double*>(take(ngroups * 8));
  s.groups_before = reinterpret_cast<double*>(take(ngroups * 8));
  s.cand_f = reinterpret_cast<double*>(take(nblocks * 8));
  s.bytes = off;
  return s;
}

}  // namespace

uint64_t optimal_scratch_bytes(uint64_t d) { return carve(nullptr, d).bytes; }

int launch_optimal_threshold(const float* row, uint64_t d, void* scratch, float* ws_threshold, float* threshold_out,
                             unsigned long long* kept_out, unsigned int* status, cudaStream_t stream) {
  const OptimalScratch s = carve(scratch, d);
  const uint32_t ntiles = static_cast<uint32_t>((d + kSortTile - 1) / kSortTile);
  const uint64_t len = static_cast<uint64_t>(kRadix) * ntiles;
  const uint32_t nchunks = static_cast<uint32_t>((len + kScanChunk - 1) / kScanChunk);
  int launches = 0;
  const uint32_t* src = reinterpret_cast<const uint32_t*>(row);
  uint32_t* dst = s.keys_a;
  for (int pass = 0; pass < kSortPasses; ++pass) {
    const uint32_t shift = pass * kRadixBits;
    if (pass == 0)
      sort_hist_kernel<true><<<ntiles, kSortThreads, 0, stream>>>(src, d, shift, ntiles, s.counts, status);
    else
      sort_hist_kernel<false><<<ntiles, kSortThreads, 0, stream>>>(src, d, shift, ntiles, s.counts, status);
    sort_scan_chunks_kernel<<<nchunks, kSortThreads, 0, stream>>>(s.counts, len, s.chunk_total);
    sort_scan_totals_kernel<<<1, kSortThreads, 0, stream>>>(s.chunk_total, nchunks);
    if (pass == 0)
      sort_scatter_kernel<true><<<ntiles, kSortThreads, 0, stream>>>(src, dst, d, shift, ntiles, s.counts, s.chunk_total);
    else
      sort_scatter_kernel<false><<<ntiles, kSortThreads, 0, stream>>>(src, dst, d, shift, ntiles, s.counts, s.chunk_total);
    launches += 4;
    src = dst;
    dst = dst == s.keys_a ? s.keys_b : s.keys_a;
  }
  const uint32_t nblocks = static_cast<uint32_t>((d + kBlock - 1) / kBlock);
  const uint32_t ngroups = (nblocks + kBlock - 1) / kBlock;
  prefix_block_totals_kernel<<<nblocks, kBlock, 0, stream>>>(src, d, s.block_total);
  prefix_group_scan_kernel<<<ngroups, kBlock, 0, stream>>>(s.block_total, nblocks, s.block_incl, s.group_total);
  prefix_groups_kernel<<<1, 32, 0, stream>>>(s.group_total, ngroups, s.groups_before);
  objective_kernel<<<nblocks, kBlock, 0, stream>>>(src, d, s.block_incl, s.groups_before, s.cand_f, s.cand_i);
  pick_kernel<<<1, kBlock, 0, stream>>>(src, d, s.cand_f, s.cand_i, nblocks, ws_threshold, threshold_out, kept_out);
  return launches + 5;
}

}  // namespace qasg

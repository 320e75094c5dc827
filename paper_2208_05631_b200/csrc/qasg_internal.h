// Internal interface between the C-ABI layer and the kernel launchers of libqasg.
#ifndef QASG_INTERNAL_H_
#define QASG_INTERNAL_H_

#include <cuda_runtime.h>
#include <stdint.h>

namespace qasg {

// Geometry of the fixed-order sums.  A tile is 4 rows x 1024 columns = 4096 consecutive
// coordinates; 256 threads own 4 adjacent columns each.
constexpr int kThreads = 256;
constexpr int kTileRows = 4;
constexpr int kTileCols = 1024;
constexpr int kTile = kTileRows * kTileCols;
// A worker's tiles are cut into at most kMaxChunks aligned groups of `group` tiles
// (group a power of two).  One CTA reduces one group to one partial; the partials of a
// worker are combined by one warp.
constexpr int kMaxChunks = 1024;
constexpr int kMaxWorkers = 64;
// The server row (the averaged gradient, re-quantized) is one long row: it may use more chunks.
constexpr int kRowChunks = 8 * kMaxChunks;
constexpr int kSelectCtasPerSm = 3;  // resident CTAs of the selection-statistics kernel

enum : unsigned { kFlagNonFinite = 1u, kFlagBadCode = 2u, kFlagBadIndex = 4u, kFlagTimeout = 8u };

struct Geometry {
  uint64_t d;       // coordinates per worker
  uint64_t ld;      // row stride of g in floats
  uint32_t M;       // workers
  uint32_t tiles;   // ceil(d / 4096)
  uint32_t group;   // tiles per chunk, power of two
  uint32_t log2_group;
  uint32_t chunks;  // ceil(tiles / group) <= kMaxChunks
};

// target_items > 0: prefer longer chunks as long as the launch keeps that many (worker, chunk) items.
Geometry make_geometry(uint64_t d, uint64_t ld, uint32_t M, uint32_t max_chunks = kMaxChunks,
                       uint32_t target_items = 0);

struct Workspace {
  double* part_sum;              // [M_max][kMaxChunks] chunk partials of a canonical sum
  uint32_t* part_max;            // [M_max][kMaxChunks] chunk maxima of |g| (bit patterns)
  unsigned long long* part_cnt;  // [M_max][kMaxChunks] chunk counts of non-zero codes
  float* thresholds;             // [M_max] Delta_m
  float* scales;                 // [M_max] s_m
  unsigned long long* counts;    // [M_max] non-zero codes
  unsigned long long* selected;  // [M_max] coordinates the worker's indicator selects (sparse selection)
  unsigned int* ticket;          // grid-completion counter, zero between launches
  unsigned int* status;          // OR of kFlag*
};

// What the CTAs of the one-launch quantizer (qasg_stream.cu) hand to one another.  Chunk partials travel
// through 64-bit slots that hold kEmptySlot until their item has stored its value; the consumer empties
// them again, so everything is back in its initial state when a call completes and a captured launch can
// be replayed.  A call that gave up leaves them in an unknown state: `abort` stays set and the host clears
// slots and words.  These arrays belong to that kernel alone.
constexpr unsigned long long kEmptySlot = 0xFFFFFFFFFFFFFFFFull;  // not the bits of any sum, count or maximum
struct StreamSlots {
  unsigned long long* sum_a;  // [M_max][kMaxChunks] chunk sums of |g| (double bits), or chunk maxima (stochastic)
  unsigned long long* sum_b;  // [M_max][kMaxChunks] chunk sums of the kept |g| (double bits)
  unsigned long long* cnt_b;  // [M_max][kMaxChunks] chunk counts of non-zero codes
};
struct StreamSync {
  unsigned int ready[kMaxWorkers];  // 1 once worker m's threshold (or scaler) of this call is published
  unsigned int abort;               // non-zero once a wait ran out: every later wait returns at once
  unsigned int probe, probe_abort;  // the wait self-test's own words (nothing ever sets probe)
  unsigned int meet_count, meet_go, meet_exit;  // the one-launch step: arrivals at its meetings, the meeting that is over, CTAs that left
};

struct StreamParams {
  float coef;            // threshold coefficient (0.75)
  uint32_t lag;          // rows between a worker's sum and its codes, 0 <= lag <= M
  uint32_t max_polls;    // bound of every wait
  uint32_t stream_base;  // Philox counter word 1 = stream_base + worker
  uint64_t seed, t;
};

struct LaunchShape {
  int sm_count;
  int reduce_ctas_per_sm;  // resident CTAs per SM for the reduction kernels
  int update_ctas_per_sm;  // same for the coordinate-wise kernels
  bool chained;            // launch the step's kernels as programmatic dependents of their predecessors
};

// Constants of the indicator test, rounded to fp32 on the host: lambda*eta, lambda*t.
struct SelectScalars {
  float lambda, lambda_t;  // QCMD compares |g| with lambda, QRDA |z + g| with lambda*t
};

struct StepScalars {
  float lambda, eta, delta, t, inv_t;
};

// Each launcher enqueues on `stream` and returns the number of kernels it launched.
// denom (device, [M]) replaces d in Delta = coef * sum / d when the sum runs over selected coordinates.
int launch_abs_sum(const float* g, const Geometry& geo, float coef, const Workspace& ws,
                   float* thresholds_out, const LaunchShape& shape, cudaStream_t stream,
                   const unsigned long long* denom = nullptr);
int launch_abs_max(const float* g, const Geometry& geo, const Workspace& ws,
                   const LaunchShape& shape, cudaStream_t stream);
int launch_threshold_codes(const float* g, const Geometry& geo, const Workspace& ws,
                           uint32_t* codes, float* scales_out, unsigned long long* counts_out,
                           const LaunchShape& shape, cudaStream_t stream, const uint32_t* indicators = nullptr);
// stream_base is added to the worker index in Philox counter word 1 (0 for workers, 1<<16 for the server row).
int launch_stochastic_codes(const float* g, const Geometry& geo, uint64_t seed, uint64_t t,
                            uint32_t stream_base, const Workspace& ws, uint32_t* codes, float* scales_out,
                            unsigned long long* counts_out, const LaunchShape& shape,
                            cudaStream_t stream, const uint32_t* indicators = nullptr);
// Sparse selection: indicators [M][ceil(d/32)] words, bit i&31 of word i>>5.
int launch_select_stats(int rule, bool stochastic, const float* g, const Geometry& geo, const float* x,
                        const float* hz, const SelectScalars& sc, float coef, const Workspace& ws,
                        uint32_t* indicators, float* thresholds_out, unsigned long long* selected_out,
                        const LaunchShape& shape, cudaStream_t stream);
int launch_indicator_or(const uint32_t* indicators, uint64_t d, uint32_t M, uint32_t* isyn,
                        unsigned long long* ksyn, const LaunchShape& shape, cudaStream_t stream);
// rule 0 = QCMD, 1 = QRDA, 2 = write the averaged gradient to x (h, z unused).
int launch_decode_update(int rule, const uint32_t* codes, const float* scales, uint64_t d,
                         uint32_t M, float* x, float* h, float* z, const StepScalars& sc,
                         unsigned int* status, const LaunchShape& shape, cudaStream_t stream);
int launch_decode_average(const uint32_t* codes, const float* scales, uint64_t d, uint32_t M,
                          float* gbar, unsigned int* status, const LaunchShape& shape,
                          cudaStream_t stream);
// Server row q = Q(average): statistics (threshold or maximum), then codes.  `row` is the geometry of
// one row of d coordinates with up to kRowChunks chunks; wsq holds kRowChunks partial slots.
int launch_avg_stats(bool stochastic, const uint32_t* codes, const float* scales, uint32_t workers,
                     const Geometry& row, float coef, const Workspace& wsq, float* threshold_out,
                     const LaunchShape& shape, cudaStream_t stream, const unsigned long long* denom = nullptr);
int launch_avg_codes(bool stochastic, const uint32_t* codes, const float* scales, uint32_t workers,
                     const Geometry& row, uint64_t seed, uint64_t t, const Workspace& wsq, uint32_t* qcodes,
                     float* scale_out, unsigned long long* count_out, const LaunchShape& shape,
                     cudaStream_t stream);
int launch_dense_update(int rule, const float* q, uint64_t d, float* x, float* h, float* z,
                        const StepScalars& sc, const LaunchShape& shape, cudaStream_t stream);
// No quantization: q = mean of the M rows of g (fp64 sum in worker order), then the update of `rule`.
int launch_mean_update(int rule, const float* g, uint64_t d, uint64_t ld, uint32_t M, float* x, float* h, float* z,
                       const StepScalars& sc, unsigned int* status, const LaunchShape& shape, cudaStream_t stream);

// margins_ws: device fp32 [M*B] scratch for the per-row coefficients.
// status: the context's flag word; row ids >= n_rows and (CSR) broken rowptr pairs or columns outside
// [0, d) are skipped and raise kFlagBadIndex.
int launch_logreg_dense(const float* X, const float* y, uint64_t n_rows, uint64_t d, uint32_t M,
                        const uint64_t* shard_row0_host, const uint32_t* batch_rows, uint32_t B,
                        uint64_t t, const float* x, float* g, uint64_t ld_g, float* coef_ws,
                        unsigned int* status, const LaunchShape& shape, cudaStream_t stream);
int launch_logreg_csr(const int64_t* rowptr, const int32_t* colidx, const float* vals,
                      const float* y, uint64_t n_rows, uint64_t d, uint32_t M, const uint64_t* shard_row0_host,
                      const uint32_t* batch_rows, uint32_t B, uint64_t t, const float* x, float* g,
                      uint64_t ld_g, unsigned int* status, const LaunchShape& shape, cudaStream_t stream,
                      uint32_t* touched = nullptr);
// With `touched` the launcher does not clear g: it adds into rows that are zero wherever the bits are zero
// and sets the bit of every entry it adds to.  launch_touched_clear re-establishes that state from the
// bits a previous gradient left: zeroes the marked entries of g, then the bits.
int launch_touched_clear(float* g, uint64_t d, uint64_t ld_g, uint32_t M, uint32_t* touched,
                         const LaunchShape& shape, cudaStream_t stream);

// Passes A and B for rows held in sparse form, one warp per tile (qasg_touched.cu): the results of the
// dense launchers on the row with +0.0 wherever a touched bit is 0.
// touched: [M][ceil(d/32)] words, bit i&31 of word i>>5; only the marked entries are stored (and read).
int launch_touched_abs_sum(const float* g, const Geometry& geo, float coef, const Workspace& ws, float* thresholds_out,
                           const uint32_t* touched, const LaunchShape& shape, cudaStream_t stream);
int launch_touched_abs_max(const float* g, const Geometry& geo, const Workspace& ws, const uint32_t* touched,
                           const LaunchShape& shape, cudaStream_t stream);
int launch_touched_codes(bool stochastic, const float* g, const Geometry& geo, uint64_t seed, uint64_t t,
                         const Workspace& ws, uint32_t* codes, float* scales_out, unsigned long long* counts_out,
                         const uint32_t* touched, const LaunchShape& shape, cudaStream_t stream);

// Exact optimal threshold of one row (rank, prefix sums, first maximum of (sum of the k largest)^2 / k).
// scratch: optimal_scratch_bytes(d) bytes of device memory, 256-byte aligned; d < 2^31.
// Writes Delta* to ws_threshold (and threshold_out, kept_out = k if not null).
uint64_t optimal_scratch_bytes(uint64_t d);
int launch_optimal_threshold(const float* row, uint64_t d, void* scratch, float* ws_threshold, float* threshold_out,
                             unsigned long long* kept_out, unsigned int* status, cudaStream_t stream);

// Passes A and B in one cooperative launch (rows that fit L2); results as launch_abs_sum/abs_max followed
// by launch_threshold_codes/stochastic_codes.  keep_codes: ordinary instead of streaming code stores.
// geo.group must not exceed kStreamMaxGroup (an item's tiles are combined in one go).
constexpr uint32_t kStreamMaxGroup = 32;
int launch_quantize_stream(bool stochastic, bool keep_codes, const float* g, const Geometry& geo,
                           const StreamParams& sp, const Workspace& ws, const StreamSlots& slots, StreamSync* sync,
                           uint32_t* codes, float* scales_out, float* thresholds_out, unsigned long long* counts_out,
                           const LaunchShape& shape, cudaStream_t stream);
// One bounded wait on a word nothing sets: raises kFlagTimeout after max_polls polls.
int launch_wait_selftest(StreamSync* sync, unsigned int* status, uint32_t max_polls, cudaStream_t stream);
// The whole fused step (passes A, B, C) as one launch whose CTAs meet twice; for small problems.
// wsb: the statistics of ws with partial slots of its own (at least [M][kMaxChunks]) for pass B.
int launch_fused_step(int rule, bool stochastic, const float* g, const Geometry& geo, float coef, uint64_t seed,
                      uint64_t t, uint32_t stream_base, uint32_t max_polls, const Workspace& ws, const Workspace& wsb,
                      StreamSync* sync, uint32_t* codes, float* scales_out, float* x, float* h, float* z,
                      const StepScalars& sc, const LaunchShape& shape, cudaStream_t stream);

void query_launch_shape(LaunchShape* shape);

}  // namespace qasg
#endif  // QASG_INTERNAL_H_

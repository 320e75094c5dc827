// qasg_quantize_pack_static: the threshold quantizer for callers that must not allocate.
//
// Everything the two quantization kernels need beyond their inputs and outputs (per-chunk
// partial sums and counts, the per-worker statistics, the grid-completion counter, the
// condition flags) lives in one file-scope device array instead of a context's workspace.
// Host code cannot use that array's name as an address: the address the kernels receive is
// obtained once per device with cudaGetSymbolAddress.
#include "../../include/qasg.h"

#include <mutex>

#include "qasg_internal.h"

using namespace qasg;

namespace {

constexpr uint32_t kStaticWorkers = QASG_STATIC_MAX_WORKERS;
constexpr int kMaxDevices = 64;

// Layout of the scratch array, in bytes from its start.
constexpr size_t kSlots = static_cast<size_t>(kStaticWorkers) * kMaxChunks;
constexpr size_t kOffPartSum = 0;
constexpr size_t kOffPartCnt = kOffPartSum + kSlots * sizeof(double);
constexpr size_t kOffPartMax = kOffPartCnt + kSlots * sizeof(unsigned long long);
constexpr size_t kOffCounts = kOffPartMax + kSlots * sizeof(uint32_t);
constexpr size_t kOffThresholds = kOffCounts + kMaxWorkers * sizeof(unsigned long long);
constexpr size_t kOffScales = kOffThresholds + kMaxWorkers * sizeof(float);
constexpr size_t kOffTicket = kOffScales + kMaxWorkers * sizeof(float);
constexpr size_t kOffStatus = kOffTicket + 256;
constexpr size_t kScratchBytes = kOffStatus + 256;
static_assert(kScratchBytes <= QASG_STATIC_SCRATCH_BYTES, "scratch layout exceeds the stated size");

// Held by every device that loads the library, until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[QASG_STATIC_SCRATCH_BYTES];

struct DeviceSetup {
  bool ready = false;
  unsigned char* scratch = nullptr;  // device address of g_static_scratch on this device
  LaunchShape shape;
};

std::mutex g_setup_mutex;
DeviceSetup g_setup[kMaxDevices];

// Once per device, with that device current: resolve the array's device address.
qasg_status setup_device(int device, DeviceSetup** out) {
  if (device < 0 || device >= kMaxDevices) return QASG_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  DeviceSetup& s = g_setup[device];
  if (!s.ready) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || ptr == nullptr) {
      cudaGetLastError();
      return QASG_ERR_CUDA;
    }
    s.scratch = static_cast<unsigned char*>(ptr);
    query_launch_shape(&s.shape);
    s.ready = true;
  }
  *out = &s;
  return QASG_OK;
}

}  // namespace

extern "C" qasg_status qasg_quantize_pack_static(int device, const float* g, uint64_t d, uint64_t ld_g,
                                                 uint32_t M, float thr_coef, uint32_t* codes, float* scales,
                                                 float* thresholds, uint64_t* counts, void* stream) {
  if (!g || !codes || !scales) return QASG_ERR_INVALID_ARG;
  if (d < 1 || d > (1ull << 34) || M < 1 || ld_g < d) return QASG_ERR_INVALID_ARG;
  if (!(thr_coef > 0.f) || !isfinite(thr_coef)) return QASG_ERR_INVALID_ARG;
  if (M > kStaticWorkers) return QASG_ERR_WORKSPACE;  // beyond what the static scratch holds
  if ((ld_g & 3u) || (reinterpret_cast<uintptr_t>(g) & 15u) || (reinterpret_cast<uintptr_t>(codes) & 15u))
    return QASG_ERR_ALIGNMENT;
  if (cudaSetDevice(device) != cudaSuccess) {
    cudaGetLastError();
    return QASG_ERR_CUDA;
  }
  DeviceSetup* s = nullptr;
  const qasg_status st = setup_device(device, &s);
  if (st != QASG_OK) return st;

  Workspace ws;
  ws.part_sum = reinterpret_cast<double*>(s->scratch + kOffPartSum);
  ws.part_cnt = reinterpret_cast<unsigned long long*>(s->scratch + kOffPartCnt);
  ws.part_max = reinterpret_cast<uint32_t*>(s->scratch + kOffPartMax);
  ws.counts = reinterpret_cast<unsigned long long*>(s->scratch + kOffCounts);
  ws.selected = nullptr;  // sparse selection is not offered by this entry point
  ws.thresholds = reinterpret_cast<float*>(s->scratch + kOffThresholds);
  ws.scales = reinterpret_cast<float*>(s->scratch + kOffScales);
  ws.ticket = reinterpret_cast<unsigned int*>(s->scratch + kOffTicket);
  ws.status = reinterpret_cast<unsigned int*>(s->scratch + kOffStatus);

  cudaStream_t cs = static_cast<cudaStream_t>(stream);
  // The array keeps what the last call left.  The completion counter and the flags must start
  // at zero; the partial slots and statistics are fully rewritten before they are read.
  if (cudaMemsetAsync(s->scratch + kOffTicket, 0, 512, cs) != cudaSuccess) {
    cudaGetLastError();
    return QASG_ERR_CUDA;
  }
  const Geometry geo = make_geometry(d, ld_g, M);
  launch_abs_sum(g, geo, thr_coef, ws, thresholds, s->shape, cs);
  launch_threshold_codes(g, geo, ws, codes, scales, reinterpret_cast<unsigned long long*>(counts), s->shape, cs);
  return cudaGetLastError() == cudaSuccess ? QASG_OK : QASG_ERR_CUDA;
}

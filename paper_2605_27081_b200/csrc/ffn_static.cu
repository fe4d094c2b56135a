// remoe_expert_ffn_static: the gate-weighted SwiGLU expert sum of one layer for callers that
// must not allocate device memory.
//
// Some embedders of this library run where cudaMalloc is off limits: inside a latency-critical
// serving loop whose memory is carved up once at start-up by another component, under a
// framework that forbids allocator calls on its worker threads, or in a process whose device
// memory is already fully committed.  The regular path allocates its scratch (per-CTA partial
// sums) when a stack is created; this entry point instead keeps that scratch in a file-scope
// device array of fixed size that is part of the loaded module, so a call performs no
// cudaMalloc, no cudaFree and no allocating library routine -- it only launches two kernels
// on the caller's stream.  The price is a fixed ceiling on the problem size and one shared
// scratch area per device.
//
// It runs the same per-CTA body as the stack's expert-streaming kernel (ffn_stream_body.cuh: channel-major
// expert block, bulk-copy stage ring fed by four producer lanes, warp-per-triple arithmetic), for one layer
// whose experts are given directly as device pointers.
#include <cuda_runtime.h>
#include <stdint.h>

#include <mutex>

#include "remoe.h"
#include "ffn_stream_body.cuh"

namespace {

using remoe::stream::kConsumerWarps;
using remoe::stream::kThreads;
constexpr int kStages = remoe::stream::kMaxStages;
constexpr int kMaxCtas = 160;                               // scratch rows; grids are capped to this
constexpr int kMaxDevices = 64;

// Scratch of the no-allocation entry point: one partial output vector per CTA.  Lives in the
// module image on every device that loads the library (1.25 MiB) until the process exits.
// Every call overwrites the rows it uses before reading them, so nothing needs clearing; two
// calls that overlap on the GPU would race on it.
static __device__ __align__(256) float g_static_partial[kMaxCtas * REMOE_STATIC_MAX_HIDDEN];

struct StaticArgs {
  const char* base[REMOE_STATIC_MAX_EXPERTS];
  float scale[REMOE_STATIC_MAX_EXPERTS];
  int prefix[REMOE_STATIC_MAX_EXPERTS + 1];                 // exclusive prefix of rows per expert
  int n_experts;
  int rows_per_cta;
  const float* hidden_in;
  float* partial;                                           // device address of g_static_partial
  int n_active;                                             // CTAs that own at least one row
};

using namespace remoe::ring;

template <int WB, int H>
constexpr size_t smem_bytes() {
  return 2 * kStages * sizeof(uint64_t) + (size_t)kConsumerWarps * 32 * (16 / WB) * sizeof(float) +
         (size_t)kStages * 3 * H * WB;
}

// One layer, experts given as pointers; one partial row per CTA in the fixed scratch array.  There is no
// error word to report through without allocating one, so a wait that ran out poisons the CTA's partial:
// the caller sees NaN in the output instead of a wrong number.
template <int H>
struct StaticWork {
  static constexpr bool kPoison = true;
  const StaticArgs& a;
  __device__ __forceinline__ const char* base(int pair, bool&) const { return a.base[pair]; }
  __device__ __forceinline__ float scale(int pair, int) const { return a.scale[pair]; }
  __device__ __forceinline__ const float* hidden(int) const { return a.hidden_in; }
  __device__ __forceinline__ float* partial(int) const { return a.partial + (size_t)blockIdx.x * H; }
  __device__ __forceinline__ void fail(int) const {}
};

template <int WB, int H>
__global__ void __launch_bounds__(kThreads, 1) ffn_static_kernel(const __grid_constant__ StaticArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + kStages;
  float* red = reinterpret_cast<float*>(smem + 2 * kStages * sizeof(uint64_t));
  unsigned char* stages = reinterpret_cast<unsigned char*>(red + kConsumerWarps * 32 * Elems<WB>::kVec);
  __shared__ int s_abort;

  if (threadIdx.x == 0) {
    s_abort = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_fence_init();
  }
  __syncthreads();

  const int M = a.prefix[a.n_experts];
  const int r0 = min(M, (int)blockIdx.x * a.rows_per_cta), r1 = min(M, r0 + a.rows_per_cta);
  if (r0 >= r1) return;

  const remoe::stream::Ring ring{full, empty, red, stages, kStages, &s_abort};
  const StaticWork<H> wk{a};
  // all experts form one "layer" of n_experts pairs
  remoe::stream::stream_rows<WB, H>(wk, a.prefix, a.n_experts, r0, r1, ring, kSpinLimit, 0);
}

__global__ void __launch_bounds__(256) combine_static_kernel(const float* __restrict__ partial, int n_active, int H,
                                                             float* __restrict__ out) {
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= H) return;
  float t = 0.f;
  for (int b = 0; b < n_active; ++b) t += partial[(size_t)b * H + c];
  out[c] = t;
}

// Per-device set-up, done by the first call on that device with that device current: resolve
// the scratch array's device address (in host code the array's name is only a stand-in for the
// symbol, not an address a kernel could use) and raise the kernels' dynamic shared-memory limit.
struct DeviceState {
  bool ready = false;
  float* scratch = nullptr;
  int sms = 0;
};
DeviceState g_dev[kMaxDevices];
std::mutex g_mu;

template <int WB, int H>
cudaError_t launch(const StaticArgs& a, int grid, cudaStream_t st) {
  ffn_static_kernel<WB, H><<<grid, kThreads, smem_bytes<WB, H>(), st>>>(a);
  return cudaGetLastError();
}

template <int WB, int H>
cudaError_t configure() {
  return cudaFuncSetAttribute(ffn_static_kernel<WB, H>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              (int)smem_bytes<WB, H>());
}

cudaError_t setup_device(int dev) {
  DeviceState& d = g_dev[dev];
  if (d.ready) return cudaSuccess;
  float* p = nullptr;
  cudaError_t e = cudaGetSymbolAddress((void**)&p, g_static_partial);
  if (e != cudaSuccess) return e;
  if ((e = cudaDeviceGetAttribute(&d.sms, cudaDevAttrMultiProcessorCount, dev)) != cudaSuccess) return e;
  if ((e = configure<4, 128>()) != cudaSuccess) return e;
  if ((e = configure<4, 256>()) != cudaSuccess) return e;
  if ((e = configure<4, 512>()) != cudaSuccess) return e;
  if ((e = configure<4, 1024>()) != cudaSuccess) return e;
  if ((e = configure<2, 256>()) != cudaSuccess) return e;
  if ((e = configure<2, 512>()) != cudaSuccess) return e;
  if ((e = configure<2, 1024>()) != cudaSuccess) return e;
  if ((e = configure<2, 2048>()) != cudaSuccess) return e;
  d.scratch = p;
  d.ready = true;
  return cudaSuccess;
}

}  // namespace

extern "C" int remoe_expert_ffn_static(int32_t hidden, int32_t weight_dtype, int32_t n_experts,
                                       const void* const* expert_blocks_dev, const int32_t* inter,
                                       const float* scales, const float* hidden_in_dev, float* hidden_out_dev,
                                       void* cuda_stream) {
  if (!expert_blocks_dev || !inter || !scales || !hidden_in_dev || !hidden_out_dev || n_experts < 1)
    return REMOE_E_ARG;
  if (weight_dtype == REMOE_FP8_E4M3 || weight_dtype == REMOE_INT4_G32) return REMOE_E_UNSUPPORTED;   // no kernel here reads these
  if (weight_dtype != REMOE_F32 && weight_dtype != REMOE_BF16) return REMOE_E_ARG;
  if (n_experts > REMOE_STATIC_MAX_EXPERTS || hidden > REMOE_STATIC_MAX_HIDDEN) return REMOE_E_UNSUPPORTED;
  const int wb = weight_dtype == REMOE_BF16 ? 2 : 4;
  const bool width_ok = wb == 4 ? (hidden == 128 || hidden == 256 || hidden == 512 || hidden == 1024)
                                : (hidden == 256 || hidden == 512 || hidden == 1024 || hidden == 2048);
  if (!width_ok) return REMOE_E_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(hidden_in_dev) | reinterpret_cast<uintptr_t>(hidden_out_dev)) & 15u)
    return REMOE_E_ARG;

  StaticArgs a{};
  a.n_experts = n_experts;
  a.prefix[0] = 0;
  for (int e = 0; e < n_experts; ++e) {
    if (!expert_blocks_dev[e] || (reinterpret_cast<uintptr_t>(expert_blocks_dev[e]) & 15u) || inter[e] < 1)
      return REMOE_E_ARG;
    if (inter[e] > REMOE_STATIC_MAX_INTER) return REMOE_E_UNSUPPORTED;
    a.base[e] = static_cast<const char*>(expert_blocks_dev[e]);
    a.scale[e] = scales[e];
    a.prefix[e + 1] = a.prefix[e] + inter[e];
  }
  a.hidden_in = hidden_in_dev;

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return REMOE_E_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return REMOE_E_UNSUPPORTED;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (setup_device(dev) != cudaSuccess) return REMOE_E_CUDA;
  }
  const DeviceState& ds = g_dev[dev];
  const int grid = ds.sms < kMaxCtas ? ds.sms : kMaxCtas;
  const int M = a.prefix[n_experts];
  a.rows_per_cta = (M + grid - 1) / grid;
  a.n_active = (M + a.rows_per_cta - 1) / a.rows_per_cta;
  a.partial = ds.scratch;
  cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);

  cudaError_t e = cudaErrorInvalidValue;
  if (wb == 4) {
    switch (hidden) {
      case 128: e = launch<4, 128>(a, grid, st); break;
      case 256: e = launch<4, 256>(a, grid, st); break;
      case 512: e = launch<4, 512>(a, grid, st); break;
      case 1024: e = launch<4, 1024>(a, grid, st); break;
    }
  } else {
    switch (hidden) {
      case 256: e = launch<2, 256>(a, grid, st); break;
      case 512: e = launch<2, 512>(a, grid, st); break;
      case 1024: e = launch<2, 1024>(a, grid, st); break;
      case 2048: e = launch<2, 2048>(a, grid, st); break;
    }
  }
  if (e != cudaSuccess) return REMOE_E_CUDA;
  combine_static_kernel<<<(hidden + 255) / 256, 256, 0, st>>>(ds.scratch, a.n_active, hidden, hidden_out_dev);
  return cudaGetLastError() == cudaSuccess ? REMOE_OK : REMOE_E_CUDA;
}

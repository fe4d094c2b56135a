// Internal declarations shared by the kernels and the host scheduler of libremoe.
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include <atomic>

#include "remoe.h"

namespace remoe {

constexpr int kMaxHidden = 2048;       // H limit: a row is at most 8 x 32 16-byte pieces; h staged in shared memory
constexpr int kMaxRouted = 256;        // N_r limit: 8 logits per lane in the top-K warp
constexpr int kMaskWords = kMaxRouted / 32;
constexpr int kMaxSlots = 256;         // C limit of the shared-memory directory image
constexpr int kMaxRequests = 1024;     // B*K limit of one layer-step
constexpr int kMaxPairs = 1024;        // L*(K+S) limit of the streaming kernel's work table
constexpr int kCounters = 6;           // tok_hits, tok_misses, uniq_hits, uniq_misses, overlap, pairs

// Device-side error codes written to DevStack::err (first writer wins).
enum : int {
  kErrNone = 0,
  kErrWaitFull = 1,     // consumer gave up waiting for a weight row
  kErrWaitEmpty = 2,    // producer gave up waiting for a free stage
  kErrBadIndex = 3,     // an expert id or slot index outside its range
  kErrDrain = 4         // copies still in flight when a kernel bailed out
};

// Everything the kernels need, passed by value.
struct DevStack {
  int L, H, N, K, I, S, Is, B, C;
  int shared_gate, renorm, wbytes;     // wbytes: bytes per expert-block element: 4 float32, 2 bfloat16, 1 fp8 e4m3;
                                       // 0 tags the 4-bit grouped format (see weight_row_bytes)
  int rbytes;                          // bytes per router / shared-gate element: 4 or 2
  int policy;
  float beta;
  int has_prev;                        // 0 on the first step after a reset
  size_t slot_bytes, shared_bytes;     // bytes of one routed / shared expert block

  const char* router;                  // [L][N][H]
  const char* shared_gate_w;           // [L][H]
  const char* shared_blocks;           // [L][S][shared_bytes]
  char* slots;                         // [L][C][slot_bytes]

  int* expert_of_slot;                 // [L][C]   -1 = empty
  int* slot_of_expert;                 // [L][N]   -1 = not resident
  unsigned long long* stamp;           // [L][C]
  unsigned* freq;                      // [L][C]
  unsigned long long* clock;           // [L]
  unsigned* prev_mask;                 // [L][B][kMaskWords]
  unsigned long long* counters;        // [L][kCounters]
  unsigned long long* load;            // [L][N]   selections per expert since the last reset

  float* shared_scale;                 // [L][B]
  int* last_overlap;                   // [L][B]   -1 when not counted
  float* last_mass;                    // [L][B]   reuse mass m_t of the last step (Eq. 2), -1 at t = 1
  double* mass_sum;                    // [L][B]   running sum of m_t over counted steps
  // Step trace, one block so that a single copy brings it to the host:
  // n_unique[L] | requests[L][B*K] | hit[L][B*K] | slot[L][B*K] | evicted[L][B*K] | depth[L][B*K]
  // | tok_hits[L]  (token-level hits of this step, App. E.2.3)
  // depth: how many of this step's experts occupied the request's slot before it within the
  // step (0 unless the step asks for more distinct experts than there are slots).
  int* trace;
  int* err;
  // Mirror of [err | trace] in mapped page-locked host memory: the resolve warp writes its layer's part
  // there as well, so the host has the miss list when the route kernel ends, with no copy on the stream.
  int* host_mirror;
  // Token groups per distinct request (batch > 1): which sequences selected it, at which rank.
  int* grp_count;                      // [L][B*K]
  int* grp_tok;                        // [L][B*K][B]
  int* grp_k;                          // [L][B*K][B]
};

// Bytes of one stored weight row of H elements: H * wbytes, or, for the 4-bit grouped format (wbytes == 0), H/2
// bytes of packed codes followed by one bfloat16 scale per group of 32 elements.
__host__ __device__ constexpr size_t weight_row_bytes(int H, int wbytes) {
  return wbytes ? (size_t)H * wbytes : (size_t)H / 2 + (size_t)H / 16;
}
// Floats that sixteen stored bytes decode to.
__host__ __device__ constexpr int weight_vec(int wbytes) { return wbytes ? 16 / wbytes : 32; }

__host__ __device__ inline int trace_ints(int L, int BK) { return 2 * L + 5 * L * BK; }
__host__ __device__ inline int* trace_tok_hits(int* t, int L, int BK) { return t + L + 5 * L * BK; }
__host__ __device__ inline int* trace_depth(int* t, int L, int BK) { return t + L + 4 * L * BK; }
__host__ __device__ inline int* trace_n_unique(int* t) { return t; }
__host__ __device__ inline int* trace_requests(int* t, int L, int BK) { return t + L; }
__host__ __device__ inline int* trace_hit(int* t, int L, int BK) { return t + L + L * BK; }
__host__ __device__ inline int* trace_slot(int* t, int L, int BK) { return t + L + 2 * L * BK; }
__host__ __device__ inline int* trace_evicted(int* t, int L, int BK) { return t + L + 3 * L * BK; }

// Streaming FFN launch description (batch 1).
struct FfnArgs {
  DevStack d;
  const float* hidden_in;              // [L][1][H]
  const float* gates;                  // [L][1][K]
  int phase;                           // 0: resident (hits + shared); 1: misses of `layer`
  int layer;                           // phase 1: the layer; phase 0: -1 = all layers, else only this one
  float* partial;                      // [2][L][grid][H]
  int* contrib;                        // [2][L][2]  (first CTA, last CTA) contributing; first > last = none
  int grid_cap;                        // CTAs per phase the partial buffer is laid out for
  unsigned spin_limit;                 // polls of one bounded wait (0 = the default limit)
  int lose_row1;                       // failure-detection test aid: the copy of row (lose_row1 - 1) of the launch's
                                       // row list is never issued, so its consumer's bounded wait runs out; 0 = none
};

// Batched (B > 1) expert kernels: tensor-core grouped GEMM over per-expert token groups.
constexpr int kMinTokTile = 8;         // smallest token tile of a batched kernel (bounds the item count)
constexpr int kUnitsPerItem = 16;      // an item's channels are cut into this many units
struct BatchArgs {
  DevStack d;
  const float* hidden_in;              // [L][B][H]
  const float* gates;                  // [L][B][K]
  int phase;                           // 0: cache hits + shared experts; 1: misses
  int layer, depth;                    // phase 0: -1 = all layers, else only this one; phase 1: which layer, which depth
  int step_id;                         // stamps the partial rows written in this step
  float* part;                         // [L][B][K+S][kUnitsPerItem][H]
  int* flags;                          // [L][B][K+S][kUnitsPerItem]
  int* plan;                           // header (8 ints) + items (4 ints each)
  int max_items;
  int tok_tile, blk_ch;                // tokens per item, channels per block (set by the launcher)
};
bool ffn_batched_supported(const DevStack& d);
cudaError_t launch_ffn_batched(const BatchArgs& a, int grid, cudaStream_t st);
// Adds the stamped partial rows of layers [layer0, layer0 + n_layers) into hidden_out[L, B, H]; with
// `chain_in` ([L + 1, B, H]) also writes chain_in[l + 1] = chain_in[l] + out[l] (residual chaining).
cudaError_t launch_combine_batched(const BatchArgs& a, float* hidden_out, int layer0, int n_layers,
                                   float* chain_in, cudaStream_t st);
// tcgen05 / TMEM variant (needs I and I_shared multiples of 64).  Its stacks keep slots and shared blocks
// in operand-tile order: a fetched block lands channel-major in a staging pool and launch_retile_tc
// rewrites it into its slot.  `maps` is an opaque, 64-byte aligned block of ffn_batched_tc_maps_bytes()
// bytes describing the staging pool, filled once per stack by ffn_batched_tc_init.
bool ffn_batched_tc_supported(const DevStack& d);
size_t ffn_batched_tc_maps_bytes();
cudaError_t ffn_batched_tc_init(const DevStack& d, const void* stage_pool, size_t stage_bytes, void* maps_out);
cudaError_t launch_ffn_batched_tc(const BatchArgs& a, int grid, cudaStream_t st);
// Rewrites n channel-major blocks of intermediate size `inter` at byte offsets src_offsets[i] of the
// staging pool (multiples of 3 * H * 2) into dst[i] in operand-tile order.  Host arrays.
cudaError_t launch_retile_tc(const DevStack& d, const void* maps, int n, const size_t* src_offsets,
                             char* const* dst, int inter, cudaStream_t st);

// Low-precision host store at batch > 1: n channel-major stored blocks at src[i] (device, 8-byte aligned) --
// src_wbytes 1: FP8 E4M3 bytes, value = byte * 2^-8; 0: the 4-bit grouped format -- are widened to bf16 and
// written to dst[i] in operand-tile order.  Host arrays.
cudaError_t launch_widen_retile_tc(const DevStack& d, int src_wbytes, int n, const void* const* src, char* const* dst,
                                   int inter, cudaStream_t st);

// Routes layers [layer0, layer0 + n_layers); `hidden_in`, `ids`, `gates` are the full [L, B, .] arrays.
cudaError_t launch_route(const DevStack& d, const float* hidden_in, int* ids, float* gates,
                         int* contrib, int layer0, int n_layers, cudaStream_t st);
cudaError_t launch_ffn_stream(const FfnArgs& a, int grid, cudaStream_t st);
// Link between two layers of the chained batch-1 step, one launch: with `do_combine` the fixed-order sum of layer
// (layer - 1)'s partials into chain_out[layer - 1] and the residual add chain_in[layer] = chain_in[layer - 1] + out;
// with `do_route` the pre-norm chain_x[layer] = rmsnorm(chain_in[layer]) and the routing of `layer` on it.
// `ticket` is one zero-initialised device word owned by the stack.
cudaError_t launch_chain_link(const DevStack& d, const FfnArgs& f, int layer, float* chain_in, float* chain_out,
                              float* chain_x, unsigned* ticket, int do_combine, int do_route, int* ids, float* gates,
                              cudaStream_t st);
// Adds the partials of layers [layer0, layer0 + n_layers) into hidden_out[L, 1, H]; with `chain_in`
// ([L + 1, 1, H]) also writes chain_in[l + 1] = chain_in[l] + out[l] (residual chaining).
cudaError_t launch_combine(const FfnArgs& a, float* hidden_out, int layer0, int n_layers, float* chain_in,
                           cudaStream_t st);
// x = h / sqrt(mean(h^2) + 1e-6) for each of `rows` [H] vectors (pre-norm of the chained mode), fixed
// summation order.
cudaError_t launch_rmsnorm(const float* h, float* x, int H, int rows, cudaStream_t st);
size_t ffn_stream_smem_bytes(int H, int wbytes, int* stages_out);

// Raises a kernel's dynamic shared-memory limit once per device (the limit is a per-device attribute of
// the kernel).  `done` is a zero-initialised array of kMaxDevices flags owned by the caller, one array per
// kernel; host threads may race here: the flags are atomic and setting the attribute twice is harmless.
constexpr int kMaxDevices = 64;
template <typename K>
inline cudaError_t allow_dynamic_smem(K kernel, size_t bytes, std::atomic<bool>* done) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  if (done[dev].load(std::memory_order_acquire)) return cudaSuccess;
  const cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) done[dev].store(true, std::memory_order_release);
  return e;
}
bool ffn_stream_supported(int H, int wbytes);

}  // namespace remoe

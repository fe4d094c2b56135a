// Streaming SwiGLU expert GEMV with fused gate-weighted combine, batch 1, sm_100a.
//
// An expert block is stored channel-major: for intermediate channel i the rows W_gate[i,:],
// W_up[i,:] and W_down[:,i] are contiguous (3*H elements).  One such triple is all the data
// needed for
//     a_i = silu(W_gate[i,:] . h) * (W_up[i,:] . h) * g          (g: gate weight / shared scale)
//     out += a_i * W_down[:, i]
// so the whole layer -- K routed experts in their cache slots plus the shared experts -- is one
// linear stream of triples with no intermediate vector in memory and no dependency between
// CTAs.  The kernel therefore treats every active (layer, expert) of the launch as one long
// row list, cuts it into equal contiguous ranges, one per CTA, and in each CTA
//   - four lanes of a producer warp move triples HBM -> shared memory with bulk async copies (TMA,
//     non-tensor form) into a ring of stages guarded by full/empty mbarriers;
//   - eight consumer warps take triples round-robin; a warp owns a whole triple: two dot
//     products by 128-bit shared loads and shuffle reduction, SiLU, then an AXPY into its
//     private fp32 copy of out[H] held in registers;
//   - at a layer boundary and at the end the eight private copies are added in a fixed order
//     and written as this CTA's partial for that layer.
// A second tiny kernel adds the partials of each layer in a fixed order (resident phase by
// ascending CTA, then miss phase by ascending CTA), so results are deterministic and no float
// atomics are used.  HBM traffic is the weight bytes once plus O(grid * H) partials.
#include "remoe_internal.cuh"
#include "tma_ring.cuh"
#include "ffn_stream_body.cuh"

namespace remoe {

namespace {

using namespace ring;
using stream::kConsumerWarps;
using stream::kMaxStages;
using stream::kThreads;

// Shared-memory carve-up (dynamic): barriers | row prefix table | reduce buffer | stage ring.
struct Layout {
  size_t bars, prefix, red, stages, total;
  int n_stages;
};
__host__ __device__ inline Layout make_layout(int H, int wbytes) {
  Layout y;
  y.bars = 0;
  y.prefix = 2 * kMaxStages * sizeof(uint64_t);
  y.red = y.prefix + (size_t)(kMaxPairs + 1) * sizeof(int);
  y.red = (y.red + 127) / 128 * 128;
  y.stages = y.red + (size_t)kConsumerWarps * 32 * weight_vec(wbytes) * sizeof(float);
  const size_t stage = 3 * weight_row_bytes(H, wbytes);
  const size_t budget = 227 * 1024 - 1024;              // leave room for static shared memory
  int n = (int)((budget - y.stages) / stage);
  n = n >= kMaxStages ? kMaxStages : (n / kConsumerWarps) * kConsumerWarps;
  y.n_stages = n;
  y.total = y.stages + (size_t)n * stage;
  return y;
}

// Rows (channel triples) a (layer, position) pair contributes to this launch.
__device__ __forceinline__ int pair_rows(const FfnArgs& a, int pair) {
  const DevStack& d = a.d;
  const int P = d.K + d.S;
  const int l = pair / P, p = pair % P;
  if (a.layer >= 0 && l != a.layer) return 0;
  if (p >= d.K) return a.phase == 0 ? d.Is : 0;
  const int hit = trace_hit(d.trace, d.L, d.K)[l * d.K + p];
  if (a.phase == 0) return hit ? d.I : 0;
  return hit ? 0 : d.I;
}

// Where a stack launch finds its rows and puts its partials: routed experts in the cache slots the step
// trace names, shared experts in their resident blocks; one partial per (phase, layer, CTA).
template <int H>
struct StackWork {
  static constexpr bool kPoison = false;
  const FfnArgs& a;
  const int* t_slot;
  __device__ __forceinline__ const char* base(int pair, bool& ok) const {
    const DevStack& d = a.d;
    const int P = d.K + d.S, l = pair / P, p = pair % P;
    if (p >= d.K) return d.shared_blocks + ((size_t)l * d.S + (p - d.K)) * d.shared_bytes;
    const int slot = t_slot[l * d.K + p];
    if (slot < 0 || slot >= d.C) { atomicCAS(d.err, kErrNone, kErrBadIndex); ok = false; return nullptr; }
    return d.slots + ((size_t)l * d.C + slot) * d.slot_bytes;
  }
  __device__ __forceinline__ float scale(int pair, int l) const {
    const int p = pair % (a.d.K + a.d.S);
    return p < a.d.K ? a.gates[l * a.d.K + p] : a.d.shared_scale[l];
  }
  __device__ __forceinline__ const float* hidden(int l) const { return a.hidden_in + (size_t)l * H; }
  __device__ __forceinline__ float* partial(int l) const {
    return a.partial + (((size_t)a.phase * a.d.L + l) * a.grid_cap + blockIdx.x) * H;
  }
  __device__ __forceinline__ void fail(int code) const { atomicCAS(a.d.err, kErrNone, code); }
};

template <int WB, int H>
__global__ void __launch_bounds__(kThreads, 1) ffn_stream_kernel(const __grid_constant__ FfnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const Layout lay = make_layout(H, WB);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + lay.bars);
  uint64_t* empty = full + kMaxStages;
  int* prefix = reinterpret_cast<int*>(smem + lay.prefix);
  const int NS = lay.n_stages;
  __shared__ int s_abort;

  const DevStack& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int P = d.K + d.S, n_pairs = d.L * P;

  // Work table: exclusive prefix of rows per pair.
  for (int i = tid; i < n_pairs; i += kThreads) prefix[i + 1] = pair_rows(a, i);
  if (tid == 0) {
    prefix[0] = 0;
    s_abort = 0;
    for (int s = 0; s < NS; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_fence_init();
  }
  __syncthreads();
  if (warp == 0) {
    int carry = 0;
    for (int base = 0; base < n_pairs; base += 32) {
      const int i = base + lane;
      int v = i < n_pairs ? prefix[i + 1] : 0;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int t = __shfl_up_sync(kFull, v, o);
        if (lane >= o) v += t;
      }
      if (i < n_pairs) prefix[i + 1] = v + carry;
      carry += __shfl_sync(kFull, v, 31);
    }
  }
  __syncthreads();

  // The row list of the launch is cut into equal contiguous ranges, one per CTA.
  const int M = prefix[n_pairs];
  const int G = gridDim.x;
  const int q = (M + G - 1) / G;                       // rows per CTA
  const int r0 = min(M, (int)blockIdx.x * q), r1 = min(M, r0 + q);

  if (blockIdx.x == 0) {
    for (int l = tid; l < d.L; l += kThreads) {
      if (a.layer >= 0 && l != a.layer) continue;
      const int lo = prefix[l * P], hi = prefix[(l + 1) * P];
      int* c = a.contrib + ((size_t)a.phase * d.L + l) * 2;
      if (hi > lo) { c[0] = lo / q; c[1] = (hi - 1) / q; } else { c[0] = 1; c[1] = 0; }
    }
  }
  if (r0 >= r1) return;

  const stream::Ring ring{full, empty, reinterpret_cast<float*>(smem + lay.red), smem + lay.stages, NS, &s_abort};
  const StackWork<H> wk{a, trace_slot(d.trace, d.L, d.K)};
  stream::stream_rows<WB, H>(wk, prefix, P, r0, r1, ring, a.spin_limit ? a.spin_limit : kSpinLimit, a.lose_row1);
}

// Fixed-order sum of a layer's per-CTA partial rows (resident phase by ascending CTA, then miss phase by ascending
// CTA).  One CTA per (256-column slice, layer): 64 threads across the slice's float4 pieces times 16 row groups; a
// thread adds the pieces of its group's rows in order, the groups are then added in order.  Splitting the rows
// over groups keeps the chain of dependent additions (and of memory round trips) 16 times shorter than one
// thread per column walking all rows.
constexpr int kCombineGroups = 16;
__global__ void __launch_bounds__(1024) combine_kernel(FfnArgs a, float* __restrict__ hidden_out, int layer0,
                                                       float* __restrict__ chain_in) {
  __shared__ float4 red[kCombineGroups][64];
  const DevStack& d = a.d;
  const int l = layer0 + blockIdx.y;
  const int c4 = threadIdx.x & 63, rg = threadIdx.x >> 6;
  const int col = blockIdx.x * 256 + c4 * 4;
  const bool active = col < d.H;
  const int* cb0 = a.contrib + ((size_t)0 * d.L + l) * 2;
  const int* cb1 = a.contrib + ((size_t)1 * d.L + l) * 2;
  const int lo0 = cb0[0], hi0 = cb0[1], lo1 = cb1[0], hi1 = cb1[1];
  const int n0 = hi0 >= lo0 ? hi0 - lo0 + 1 : 0, n1 = hi1 >= lo1 ? hi1 - lo1 + 1 : 0;
  const int n = n0 + n1, per = (n + kCombineGroups - 1) / kCombineGroups;
  const int ra = min(n, rg * per), rb = min(n, ra + per);
  float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
  if (active) {
    const float* p0 = a.partial + ((size_t)(0 * d.L + l) * a.grid_cap) * d.H + col;
    const float* p1 = a.partial + ((size_t)(1 * d.L + l) * a.grid_cap) * d.H + col;
#pragma unroll 8
    for (int r = ra; r < rb; ++r) {
      const float* src = r < n0 ? p0 + (size_t)(lo0 + r) * d.H : p1 + (size_t)(lo1 + r - n0) * d.H;
      const float4 v = __ldg(reinterpret_cast<const float4*>(src));
      t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
    }
  }
  red[rg][c4] = t;
  __syncthreads();
  if (rg != 0 || !active) return;
  float4 o = red[0][c4];
#pragma unroll
  for (int g = 1; g < kCombineGroups; ++g) { o.x += red[g][c4].x; o.y += red[g][c4].y; o.z += red[g][c4].z; o.w += red[g][c4].w; }
  *reinterpret_cast<float4*>(hidden_out + (size_t)l * d.H + col) = o;
  if (chain_in) {
    const float4 hp = *reinterpret_cast<const float4*>(chain_in + (size_t)l * d.H + col);
    *reinterpret_cast<float4*>(chain_in + (size_t)(l + 1) * d.H + col) =
        make_float4(hp.x + o.x, hp.y + o.y, hp.z + o.z, hp.w + o.w);
  }
}

__global__ void __launch_bounds__(256) rmsnorm_kernel(const float* __restrict__ h_all, float* __restrict__ x_all,
                                                      int H) {
  __shared__ float warp_ss[8];
  __shared__ float s_scale;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const float* h = h_all + (size_t)blockIdx.x * H;
  float* x = x_all + (size_t)blockIdx.x * H;
  float ss = 0.f;
  for (int c = tid; c < H; c += 256) ss = fmaf(h[c], h[c], ss);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(kFull, ss, o);
  if (lane == 0) warp_ss[warp] = ss;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += warp_ss[w];
    s_scale = rsqrtf(t / (float)H + 1e-6f);
  }
  __syncthreads();
  for (int c = tid; c < H; c += 256) x[c] = h[c] * s_scale;
}

template <int WB, int H>
cudaError_t launch_one(const FfnArgs& a, int grid, cudaStream_t st) {
  const Layout lay = make_layout(H, WB);
  static std::atomic<bool> configured[kMaxDevices];
  const cudaError_t e = allow_dynamic_smem(ffn_stream_kernel<WB, H>, lay.total, configured);
  if (e != cudaSuccess) return e;
  ffn_stream_kernel<WB, H><<<grid, kThreads, lay.total, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

bool ffn_stream_supported(int H, int wbytes) {
  if (wbytes == 0) return H == 1024 || H == 2048;
  if (wbytes == 4) return H == 128 || H == 256 || H == 512 || H == 1024;
  if (wbytes == 2) return H == 256 || H == 512 || H == 1024 || H == 2048;
  if (wbytes == 1) return H == 512 || H == 1024 || H == 2048;
  return false;
}

size_t ffn_stream_smem_bytes(int H, int wbytes, int* stages_out) {
  const Layout lay = make_layout(H, wbytes);
  if (stages_out) *stages_out = lay.n_stages;
  return lay.total;
}

cudaError_t launch_ffn_stream(const FfnArgs& a, int grid, cudaStream_t st) {
  const int H = a.d.H;
  if (a.d.wbytes == 4) {
    switch (H) {
      case 128: return launch_one<4, 128>(a, grid, st);
      case 256: return launch_one<4, 256>(a, grid, st);
      case 512: return launch_one<4, 512>(a, grid, st);
      case 1024: return launch_one<4, 1024>(a, grid, st);
    }
  } else if (a.d.wbytes == 2) {
    switch (H) {
      case 256: return launch_one<2, 256>(a, grid, st);
      case 512: return launch_one<2, 512>(a, grid, st);
      case 1024: return launch_one<2, 1024>(a, grid, st);
      case 2048: return launch_one<2, 2048>(a, grid, st);
    }
  } else if (a.d.wbytes == 1) {
    switch (H) {
      case 512: return launch_one<1, 512>(a, grid, st);
      case 1024: return launch_one<1, 1024>(a, grid, st);
      case 2048: return launch_one<1, 2048>(a, grid, st);
    }
  } else {
    switch (H) {
      case 1024: return launch_one<0, 1024>(a, grid, st);
      case 2048: return launch_one<0, 2048>(a, grid, st);
    }
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_rmsnorm(const float* h, float* x, int H, int rows, cudaStream_t st) {
  rmsnorm_kernel<<<rows, 256, 0, st>>>(h, x, H);
  return cudaGetLastError();
}

cudaError_t launch_combine(const FfnArgs& a, float* hidden_out, int layer0, int n_layers, float* chain_in,
                           cudaStream_t st) {
  dim3 grid((a.d.H + 255) / 256, n_layers);
  combine_kernel<<<grid, 1024, 0, st>>>(a, hidden_out, layer0, chain_in);
  return cudaGetLastError();
}

}  // namespace remoe

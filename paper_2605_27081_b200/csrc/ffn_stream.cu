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

namespace remoe {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 16;                 // multiple of kConsumerWarps
constexpr int kProducerLanes = 4;              // divides kConsumerWarps, hence every ring depth
using namespace ring;

// Shared-memory carve-up (dynamic): barriers | row prefix table | reduce buffer | stage ring.
// The ring depth is a multiple of the consumer-warp count, so a stage is always consumed by
// the same warp.  That warp has waited for fill k-1 of the stage before it waits for fill k,
// hence the barrier can never be a whole phase behind the parity it is asked about (a parity
// wait cannot tell "phase k done" from "phase k-2 done").
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

template <int WB, int H>
__global__ void __launch_bounds__(kThreads, 1) ffn_stream_kernel(const __grid_constant__ FfnArgs a) {
  using E = Elems<WB>;
  constexpr int kVec = E::kVec;
  constexpr int kIter = H / (32 * kVec);
  constexpr int kCols = kIter * kVec;                  // columns of h / out owned by one lane
  constexpr uint32_t kRowBytes = (uint32_t)weight_row_bytes(H, WB);
  constexpr uint32_t kStageBytes = 3u * kRowBytes;
  constexpr bool kGrouped = WB == 0;                   // per-group scales follow the codes of a row

  extern __shared__ __align__(128) unsigned char smem[];
  const Layout lay = make_layout(H, WB);
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + lay.bars);
  uint64_t* empty = full + kMaxStages;
  int* prefix = reinterpret_cast<int*>(smem + lay.prefix);
  float* red = reinterpret_cast<float*>(smem + lay.red);
  unsigned char* stages = smem + lay.stages;
  const int NS = lay.n_stages;
  __shared__ int s_abort;

  const DevStack& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int P = d.K + d.S, n_pairs = d.L * P;
  const unsigned spin = a.spin_limit ? a.spin_limit : kSpinLimit;

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

  const int* t_slot = trace_slot(d.trace, d.L, d.K);

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    // Issuing one copy (free-stage wait, expect_tx, bulk copy) is a chain of a few hundred cycles for one
    // thread; with small stages (FP8, narrow H) a single issuer cannot keep the ring full, so a few
    // lanes issue side by side, lane j taking the rows whose local index is j modulo kProducerLanes.
    if (lane < kProducerLanes) {
      int pair = 0;
      const char* base = nullptr;
      int pair_of_base = -1;
      int issued = lane;                             // local index after this lane's last issued row
      bool ok = true;
      for (int r = r0 + lane; r < r1 && ok; r += kProducerLanes, issued += kProducerLanes) {
        while (prefix[pair + 1] <= r) ++pair;
        if (pair != pair_of_base) {
          const int l = pair / P, p = pair % P;
          if (p < d.K) {
            const int slot = t_slot[l * d.K + p];
            if (slot < 0 || slot >= d.C) { atomicCAS(d.err, kErrNone, kErrBadIndex); ok = false; break; }
            base = d.slots + ((size_t)l * d.C + slot) * d.slot_bytes;
          } else {
            base = d.shared_blocks + ((size_t)l * d.S + (p - d.K)) * d.shared_bytes;
          }
          pair_of_base = pair;
        }
        const int i = r - prefix[pair];
        const int n = r - r0, s = n % NS;
        if (n >= NS) {
          if (*(volatile int*)&s_abort) { ok = false; break; }
          if (!mbar_wait(empty + s, ((n / NS) - 1) & 1, spin)) {
            atomicCAS(d.err, kErrNone, kErrWaitEmpty);
            ok = false;
            break;
          }
        }
        if (r + 1 == a.lose_row1) continue;                // test aid: this stage is never filled
        mbar_expect_tx(full + s, kStageBytes);
        bulk_g2s(stages + (size_t)s * kStageBytes, base + (size_t)i * kStageBytes, kStageBytes, full + s);
      }
      if (!ok || *(volatile int*)&s_abort) {
        // Let the consumers leave, then wait (bounded) for copies that are still landing.
        atomicExch(&s_abort, 1);
        for (int n = issued - kProducerLanes; n >= 0 && n >= issued - NS; n -= kProducerLanes)
          if (!mbar_wait(full + (n % NS), (n / NS) & 1, spin)) atomicCAS(d.err, kErrNone, kErrDrain);
      }
    }
  } else {
    // ----------------------------------------------------------------- consumers
    float hreg[kCols], acc[kCols];
    int pair = 0;
    while (prefix[pair + 1] <= r0) ++pair;
    int l_first = pair / P;
    int pair_last = pair;
    while (prefix[pair_last + 1] < r1) ++pair_last;
    const int l_last = pair_last / P;
    bool aborted = false;

    for (int l = l_first; l <= l_last; ++l) {
      const int lo = max(r0, prefix[l * P]), hi = min(r1, prefix[(l + 1) * P]);
      if (lo >= hi) continue;
      const float* h = a.hidden_in + (size_t)l * H;
#pragma unroll
      for (int it = 0; it < kIter; ++it) {
#pragma unroll
        for (int v4 = 0; v4 < kVec / 4; ++v4) {
          const float4 x = __ldg(reinterpret_cast<const float4*>(h + (it * 32 + lane) * kVec) + v4);
          hreg[it * kVec + v4 * 4 + 0] = x.x;
          hreg[it * kVec + v4 * 4 + 1] = x.y;
          hreg[it * kVec + v4 * 4 + 2] = x.z;
          hreg[it * kVec + v4 * 4 + 3] = x.w;
        }
      }
#pragma unroll
      for (int c = 0; c < kCols; ++c) acc[c] = 0.f;

      // first row of this layer handled by this warp: local index n = r - r0 with n % 8 == warp
      int r = lo + ((warp - (lo - r0)) % kConsumerWarps + kConsumerWarps) % kConsumerWarps;
      float scale = 0.f;
      int pair_of_scale = -1;
      for (; r < hi && !aborted; r += kConsumerWarps) {
        while (prefix[pair + 1] <= r) ++pair;
        if (pair != pair_of_scale) {
          const int p = pair % P;
          scale = p < d.K ? a.gates[l * d.K + p] : d.shared_scale[l];
          pair_of_scale = pair;
        }
        const int n = r - r0, s = n % NS;
        // decided for the whole warp: the shuffles below need every lane
        if (__any_sync(kFull, *(volatile int*)&s_abort || !mbar_wait(full + s, (n / NS) & 1, spin))) {
          if (!*(volatile int*)&s_abort) { atomicCAS(d.err, kErrNone, kErrWaitFull); atomicExch(&s_abort, 1); }
          aborted = true;
          break;
        }
        const char* st = reinterpret_cast<const char*>(stages) + (size_t)s * kStageBytes;
        float g = 0.f, u = 0.f;
        float gs[kGrouped ? kIter : 1];                  // grouped format: this lane's group scales of the third row
        if constexpr (kGrouped) {
#pragma unroll
          for (int it = 0; it < kIter; ++it) {
            float w[kVec], t = 0.f;
            E::load(st + (it * 32 + lane) * 16, w);
#pragma unroll
            for (int j = 0; j < kVec; ++j) t = fmaf(w[j], hreg[it * kVec + j], t);
            g = fmaf(E::scale(st, H, it * 32 + lane), t, g);
          }
#pragma unroll
          for (int it = 0; it < kIter; ++it) {
            float w[kVec], t = 0.f;
            E::load(st + kRowBytes + (it * 32 + lane) * 16, w);
#pragma unroll
            for (int j = 0; j < kVec; ++j) t = fmaf(w[j], hreg[it * kVec + j], t);
            u = fmaf(E::scale(st + kRowBytes, H, it * 32 + lane), t, u);
            gs[it] = E::scale(st + 2 * kRowBytes, H, it * 32 + lane);
          }
        } else {
#pragma unroll
          for (int it = 0; it < kIter; ++it) {
            float w[kVec];
            E::load(st + (it * 32 + lane) * 16, w);
#pragma unroll
            for (int j = 0; j < kVec; ++j) g = fmaf(w[j], hreg[it * kVec + j], g);
          }
#pragma unroll
          for (int it = 0; it < kIter; ++it) {
            float w[kVec];
            E::load(st + kRowBytes + (it * 32 + lane) * 16, w);
#pragma unroll
            for (int j = 0; j < kVec; ++j) u = fmaf(w[j], hreg[it * kVec + j], u);
          }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          g += __shfl_xor_sync(kFull, g, o);
          u += __shfl_xor_sync(kFull, u, o);
        }
        g *= WScale<WB>::kDot;
        u *= WScale<WB>::kDot;
        const float av = g / (1.f + __expf(-g)) * u * scale * WScale<WB>::kAct;
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
          float w[kVec];
          E::load(st + 2 * kRowBytes + (it * 32 + lane) * 16, w);
          const float a_it = kGrouped ? av * gs[kGrouped ? it : 0] : av;
#pragma unroll
          for (int j = 0; j < kVec; ++j) acc[it * kVec + j] = fmaf(a_it, w[j], acc[it * kVec + j]);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(empty + s);
      }

      // Layer flush: add the eight private copies in warp order, write this CTA's partial.
      // One pass per 32*kVec columns keeps the exchange buffer at a few KB.
      float* dst = a.partial + (((size_t)a.phase * d.L + l) * a.grid_cap + blockIdx.x) * H;
      constexpr int kPassCols = 32 * kVec;
#pragma unroll
      for (int it = 0; it < kIter; ++it) {
        float* mine = red + (size_t)warp * kPassCols + lane * kVec;
#pragma unroll
        for (int v4 = 0; v4 < kVec / 4; ++v4)
          *reinterpret_cast<float4*>(mine + v4 * 4) =
              make_float4(acc[it * kVec + v4 * 4], acc[it * kVec + v4 * 4 + 1],
                          acc[it * kVec + v4 * 4 + 2], acc[it * kVec + v4 * 4 + 3]);
        consumer_bar();
        for (int c = tid; c < kPassCols; c += kConsumerWarps * 32) {
          float t = 0.f;
#pragma unroll
          for (int w = 0; w < kConsumerWarps; ++w) t += red[(size_t)w * kPassCols + c];
          dst[it * kPassCols + c] = t;
        }
        consumer_bar();
      }
    }
  }
}

__global__ void __launch_bounds__(256) combine_kernel(FfnArgs a, float* __restrict__ hidden_out, int layer0,
                                                      float* __restrict__ chain_in) {
  const DevStack& d = a.d;
  const int l = layer0 + blockIdx.y;
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= d.H) return;
  float t = 0.f;
  for (int phase = 0; phase < 2; ++phase) {
    const int* cb = a.contrib + ((size_t)phase * d.L + l) * 2;
    const int lo = cb[0], hi = cb[1];
    const float* p = a.partial + (((size_t)phase * d.L + l) * a.grid_cap) * d.H + c;
    for (int b = lo; b <= hi; ++b) t += p[(size_t)b * d.H];
  }
  hidden_out[(size_t)l * d.H + c] = t;
  if (chain_in) chain_in[(size_t)(l + 1) * d.H + c] = chain_in[(size_t)l * d.H + c] + t;
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
  combine_kernel<<<grid, 256, 0, st>>>(a, hidden_out, layer0, chain_in);
  return cudaGetLastError();
}

}  // namespace remoe

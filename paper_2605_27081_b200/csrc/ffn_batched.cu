// Batched expert step (B > 1): tensor-core grouped GEMM over per-expert token groups, sm_100a.
//
// Tokens are grouped per requested expert (App. E.2.3: the step's distinct requests U); a work
// item is (layer, expert, tile of up to 8 of its tokens).  For an item the expert's channel-major
// block is streamed once, eight channels (24 rows) per stage, by bulk async copies into a
// two-stage shared-memory ring (rows padded by 16 bytes so that ldmatrix is conflict free).
// Eight consumer warps share every stage; warp w owns columns [256w/8.., ) of H -- the same slice
// for both contractions:
//   1. [W_gate rows; W_up rows] (16 x H_slice, A operand by ldmatrix) times X (H_slice x 8 tokens,
//      B operand held in registers as bf16) -> partial gate/up pre-activations, mma m16n8k16;
//      the eight K-slices are added through shared memory (double buffered, one barrier/stage);
//   2. a = silu(g) * u * gate weight, rounded to bf16, is the B operand (8 channels x 8 tokens)
//      of W_down^T (H_slice x 8 channels, A operand by ldmatrix.trans) -> mma m16n8k8 into fp32
//      accumulators out[H_slice x 8 tokens] kept in registers for the whole item.
// Items are laid end to end in units (1/16 of an item's channels); each CTA takes an equal
// contiguous range of units and writes one partial row per (token, expert) and piece, stamped
// with the step number; a combine kernel adds a token's stamped rows in a fixed order.  No float
// atomics; every wait is bounded.
#include "remoe_internal.cuh"
#include "tma_ring.cuh"
#include "batched_plan.cuh"

namespace remoe {

namespace {

constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kStages = 2;
constexpr int kBlockCh = 8;                           // channels per stage
constexpr int kTokTile = 8;                           // tokens per work item (the MMA's N)
constexpr int kBarBytes = 128;                        // barrier area at the start of shared memory
using namespace ring;

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(addr));
}
__device__ __forceinline__ void mma_k16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void mma_k8(float* c, uint32_t a0, uint32_t a1, uint32_t b0) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5}, {%6}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(b0));
}
// two floats -> packed bf16 pair (lo in the low half), round to nearest even
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// ------------------------------------------------------------------------------- kernel

template <int H>
struct Geo {
  static constexpr int kRowStride = H * 2 + 16;                        // padded bf16 row
  static constexpr int kStageBytes = 3 * kBlockCh * kRowStride;
  static constexpr uint32_t kTxBytes = 3u * kBlockCh * H * 2;
  static constexpr int kSlice = H / kConsumerWarps;                    // columns of H per warp
  static constexpr int kKSteps = kSlice / 16;
  static constexpr int kMTiles = kSlice / 16;
  static constexpr size_t kRedBytes = 2 * kConsumerWarps * 16 * 8 * sizeof(float);
  static constexpr size_t kSmem = kBarBytes + kRedBytes + (size_t)kStages * kStageBytes;
};

template <int H>
__global__ void __launch_bounds__(kThreads, 1) ffn_batched_kernel(const __grid_constant__ BatchArgs a) {
  using G = Geo<H>;
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem);
  uint64_t* empty = full + kStages;
  float* red = reinterpret_cast<float*>(smem + kBarBytes);
  unsigned char* stages = reinterpret_cast<unsigned char*>(red) + G::kRedBytes;
  __shared__ int s_abort;

  const DevStack& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int BK = d.B * d.K, P = d.K + d.S;
  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < kStages; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, kConsumerWarps); }
    mbar_fence_init();
  }
  __syncthreads();

  const int n_items = a.plan[0], n_units = a.plan[1];
  const int q = (n_units + gridDim.x - 1) / (int)gridDim.x;
  const int ua = min(n_units, (int)blockIdx.x * q), ub = min(n_units, ua + q);
  if (ua >= ub) return;
  const int j0 = first_item(a, n_items, ua);

  if (warp == kConsumerWarps) {
    // ------------------------------------------------------------------ producer
    // The whole warp walks the work list; lane 0 waits for the free stage and posts the byte count,
    // then the stage's 24 row copies are issued by 24 lanes side by side (issued by one thread they
    // take most of the time the stage's bytes need on the memory system).
    int n = 0;
    bool ok = true;
    for (int j = j0; j < n_items && ok; ++j) {
      if (a.plan[kPlanHeader + 4 * j + 3] >= ub) break;
      PieceInfo p;
      if (!make_piece(a, j, ua, ub, p)) continue;
      for (int blk = p.blk0; blk < p.blk1; ++blk, ++n) {
        const int s = n % kStages;
        int go = 1;
        if (lane == 0) {
          if (n >= kStages && (*(volatile int*)&s_abort || !mbar_wait(empty + s, ((n / kStages) - 1) & 1))) {
            if (!*(volatile int*)&s_abort) atomicCAS(d.err, kErrNone, kErrWaitEmpty);
            go = 0;
          } else {
            mbar_expect_tx(full + s, G::kTxBytes);
          }
        }
        go = __shfl_sync(kFull, go, 0);
        if (!go) { ok = false; break; }
        const char* src = p.base + (size_t)blk * (3 * kBlockCh * H * 2);
        unsigned char* dst = stages + (size_t)s * G::kStageBytes;
        if (lane < 3 * kBlockCh) bulk_g2s(dst + lane * G::kRowStride, src + (size_t)lane * H * 2, H * 2, full + s);
      }
    }
    __syncwarp();
    if (!ok && lane == 0) {
      atomicExch(&s_abort, 1);
      for (int m = max(0, n - kStages); m < n; ++m)
        if (!mbar_wait(full + (m % kStages), (m / kStages) & 1)) atomicCAS(d.err, kErrNone, kErrDrain);
    }
    return;
  }

  // ------------------------------------------------------------------- consumers
  const int col0 = warp * G::kSlice;                 // this warp's slice of H
  const int grp = lane >> 2, qd = lane & 3;          // MMA fragment coordinates
  int n = 0, buf = 0;
  bool aborted = false;
  for (int j = j0; j < n_items; ++j) {
    if (a.plan[kPlanHeader + 4 * j + 3] >= ub) break;
    PieceInfo p;
    if (!make_piece(a, j, ua, ub, p)) continue;

    // token metadata: B-operand column `grp` is token grp of the tile; accumulator columns are
    // tokens 2*qd and 2*qd+1.
    const int gidx = (p.l * BK + p.cand) * d.B + p.tile * kTokTile;
    auto tok_of = [&](int t) -> int {
      if (t >= p.n_tok) return -1;
      return p.shared ? p.tile * kTokTile + t : d.grp_tok[gidx + t];
    };
    auto kq_of = [&](int t) -> int { return p.shared ? d.K + (p.cand - BK) : d.grp_k[gidx + t]; };
    const int my_tok = tok_of(grp);
    float my_scale = 0.f;
    if (my_tok >= 0)
      my_scale = p.shared ? d.shared_scale[p.l * d.B + my_tok] : a.gates[((size_t)p.l * d.B + my_tok) * d.K + kq_of(grp)];

    // X slice as B fragments: for k-step ks, b0 = X[col0+16ks+2qd .. +1][tok grp], b1 = same +8.
    uint32_t xb[G::kKSteps][2];
    {
      const float* xr = my_tok >= 0 ? a.hidden_in + ((size_t)p.l * d.B + my_tok) * H + col0 : nullptr;
#pragma unroll
      for (int ks = 0; ks < G::kKSteps; ++ks) {
        float2 lo = make_float2(0.f, 0.f), hi = make_float2(0.f, 0.f);
        if (xr) {
          lo = __ldg(reinterpret_cast<const float2*>(xr + 16 * ks + 2 * qd));
          hi = __ldg(reinterpret_cast<const float2*>(xr + 16 * ks + 8 + 2 * qd));
        }
        xb[ks][0] = pack_bf16(lo.x, lo.y);
        xb[ks][1] = pack_bf16(hi.x, hi.y);
      }
    }
    float acc[G::kMTiles][4];
#pragma unroll
    for (int m = 0; m < G::kMTiles; ++m) { acc[m][0] = acc[m][1] = acc[m][2] = acc[m][3] = 0.f; }

    for (int blk = p.blk0; blk < p.blk1 && !aborted; ++blk, ++n) {
      const int s = n % kStages;
      // warp-uniform, because the tensor-core instructions below need the whole warp
      const bool fail = __any_sync(kFull, *(volatile int*)&s_abort || !mbar_wait(full + s, (n / kStages) & 1));
      const uint32_t st = smem_u32(stages + (size_t)s * G::kStageBytes);
      // contraction 1 over this warp's K slice: rows 0-7 = W_gate, rows 8-15 = W_up of the block
      if (!fail) {
        float c1[4] = {0.f, 0.f, 0.f, 0.f};
        const int mat = lane >> 3, r = lane & 7;
        const uint32_t row_addr = st + (3 * r + (mat & 1)) * G::kRowStride + (col0 + 8 * (mat >> 1)) * 2;
#pragma unroll
        for (int ks = 0; ks < G::kKSteps; ++ks) {
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4(row_addr + ks * 32, a0, a1, a2, a3);
          mma_k16(c1, a0, a1, a2, a3, xb[ks][0], xb[ks][1]);
        }
        float* rb = red + (size_t)buf * kConsumerWarps * 128 + warp * 128;
        *reinterpret_cast<float2*>(rb + grp * 8 + 2 * qd) = make_float2(c1[0], c1[1]);
        *reinterpret_cast<float2*>(rb + (grp + 8) * 8 + 2 * qd) = make_float2(c1[2], c1[3]);
      }
      if (consumer_bar_any(fail)) {
        // some warp's wait ran out (or the producer gave up): everybody leaves together
        if (tid == 0) { atomicCAS(d.err, kErrNone, kErrWaitFull); atomicExch(&s_abort, 1); }
        aborted = true;
        break;
      }
      // full pre-activations for channels 2qd, 2qd+1 and token grp, then the activation
      uint32_t ab;
      {
        const float* r0 = red + (size_t)buf * kConsumerWarps * 128;
        float g0 = 0.f, g1 = 0.f, u0 = 0.f, u1 = 0.f;
#pragma unroll
        for (int w = 0; w < kConsumerWarps; ++w) {
          g0 += r0[w * 128 + (2 * qd) * 8 + grp];
          g1 += r0[w * 128 + (2 * qd + 1) * 8 + grp];
          u0 += r0[w * 128 + (8 + 2 * qd) * 8 + grp];
          u1 += r0[w * 128 + (9 + 2 * qd) * 8 + grp];
        }
        const float v0 = g0 / (1.f + __expf(-g0)) * u0 * my_scale;
        const float v1 = g1 / (1.f + __expf(-g1)) * u1 * my_scale;
        ab = pack_bf16(v0, v1);
      }
      // contraction 2: out[H slice x 8 tokens] += W_down[:, block]^T (8 channels) x a
      {
        const int mat = lane >> 3, r = lane & 7;
        const uint32_t row_addr = st + (3 * r + 2) * G::kRowStride + (col0 + 8 * mat) * 2;
#pragma unroll
        for (int mp = 0; mp < G::kMTiles / 2; ++mp) {
          uint32_t a0, a1, a2, a3;
          ldmatrix_x4_trans(row_addr + mp * 64, a0, a1, a2, a3);
          mma_k8(acc[2 * mp], a0, a1, ab);
          mma_k8(acc[2 * mp + 1], a2, a3, ab);
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty + s);
      buf ^= 1;
    }

    // flush: one stamped partial row per (token, expert rank) for this piece
    if (!aborted) {
#pragma unroll
      for (int tt = 0; tt < 2; ++tt) {
        const int t = 2 * qd + tt;
        const int tok = tok_of(t);
        if (tok < 0) continue;
        const size_t row = (((size_t)p.l * d.B + tok) * P + kq_of(t)) * kUnitsPerItem + p.first_unit;
        float* dst = a.part + row * H + col0;
#pragma unroll
        for (int m = 0; m < G::kMTiles; ++m) {
          dst[16 * m + grp] = acc[m][tt];
          dst[16 * m + 8 + grp] = acc[m][2 + tt];
        }
        if (warp == 0 && grp == 0) a.flags[row] = a.step_id;
      }
    }
  }
}

__global__ void __launch_bounds__(256) combine_batched_kernel(BatchArgs a, float* __restrict__ hidden_out,
                                                              int layer0, float* __restrict__ chain_in) {
  const DevStack& d = a.d;
  const int lb = layer0 * d.B + blockIdx.y;
  const int c = blockIdx.x * 256 + threadIdx.x;
  if (c >= d.H) return;
  const int P = d.K + d.S;
  float t = 0.f;
  for (int k = 0; k < P; ++k)
    for (int u = 0; u < kUnitsPerItem; ++u) {
      const size_t row = ((size_t)lb * P + k) * kUnitsPerItem + u;
      if (a.flags[row] == a.step_id) t += a.part[row * d.H + c];
    }
  hidden_out[(size_t)lb * d.H + c] = t;
  if (chain_in) chain_in[((size_t)lb + d.B) * d.H + c] = chain_in[(size_t)lb * d.H + c] + t;
}

template <int H>
cudaError_t launch_one(const BatchArgs& a, int grid, cudaStream_t st) {
  static std::atomic<bool> configured[kMaxDevices];
  cudaError_t e0 = allow_dynamic_smem(ffn_batched_kernel<H>, Geo<H>::kSmem, configured);
  if (e0 != cudaSuccess) return e0;
  BatchArgs b = a;
  b.tok_tile = kTokTile;
  b.blk_ch = kBlockCh;
  plan_kernel<<<1, 1024, 0, st>>>(b);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ffn_batched_kernel<H><<<grid, kThreads, Geo<H>::kSmem, st>>>(b);
  return cudaGetLastError();
}

}  // namespace

bool ffn_batched_supported(const DevStack& d) {
  if (d.wbytes != 2) return false;
  if (d.H != 256 && d.H != 512 && d.H != 1024 && d.H != 2048) return false;
  if (d.I % kBlockCh || (d.S && d.Is % kBlockCh)) return false;
  return true;
}

cudaError_t launch_ffn_batched(const BatchArgs& a, int grid, cudaStream_t st) {
  switch (a.d.H) {
    case 256: return launch_one<256>(a, grid, st);
    case 512: return launch_one<512>(a, grid, st);
    case 1024: return launch_one<1024>(a, grid, st);
    case 2048: return launch_one<2048>(a, grid, st);
  }
  return cudaErrorInvalidValue;
}

cudaError_t launch_combine_batched(const BatchArgs& a, float* hidden_out, int layer0, int n_layers,
                                   float* chain_in, cudaStream_t st) {
  dim3 grid((a.d.H + 255) / 256, n_layers * a.d.B);
  combine_batched_kernel<<<grid, 256, 0, st>>>(a, hidden_out, layer0, chain_in);
  return cudaGetLastError();
}

}  // namespace remoe

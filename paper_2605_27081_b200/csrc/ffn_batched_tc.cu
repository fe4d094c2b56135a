// Batched expert step on the fifth-generation tensor cores (tcgen05 / TMEM), sm_100a.
//
// Same work list as ffn_batched.cu, with a work item of (layer, expert, tile of up to 16 tokens)
// and channel blocks of 64.  Per CTA (one per SM, 192 threads):
//   warp 4   TMA producer: one bulk copy (cp.async.bulk, per CTA) per 16 KB operand tile into a
//            shared-memory ring.  Slots and shared blocks of such a stack are kept in OPERAND-TILE
//            ORDER: per 64-channel group the H/64 A1 tiles, then the H/128 A2 tiles, each stored as
//            the 128-byte-swizzled image the tensor cores read, so a tile is one contiguous 16 KB run
//            in HBM (row pieces of 128 bytes at a 4 KB pitch cost about 5 % of the DRAM rate):
//              A1 tile  = [64 channels x {gate, up}] x 64 columns of H   (K-major, 128 rows)
//              A2 tile  = 64 channels x 128 columns of W_down             (MN-major, two halves)
//            retile_kernel below produces that order from a freshly fetched channel-major block with
//            tensor-map loads (cp.async.bulk.tensor, 128-byte swizzle) and bulk stores.
//   warp 5   one elected thread issues tcgen05.mma (M = 128, N = 16, K = 16, bf16 -> fp32):
//              D1[128 x 16]        += A1(kc) . X^T(kc)        for the H/64 column chunks
//              D2[ht][128 x 16]    += A2(ht)^T . a            for the H/128 output tiles
//            and releases ring stages / signals the other warps with tcgen05.commit;
//   warps 0-3  stage the token tile's hidden states as the bf16 B operand X^T (swizzled by hand),
//            read D1 from TMEM (tcgen05.ld; gate and up rows of a channel sit in neighbouring
//            lanes), form a = silu(g) * u * gate weight in bf16 as the second B operand, and at
//            the end of a piece read D2 and write one stamped partial row per (token, rank).
// The first contraction of group g+1 is issued before the second contraction of group g (D1 is
// double buffered), so the tensor pipe and the weight stream never wait for the activation step.
// Accumulators live in TMEM: D1 in 2 x 16 columns, D2 in 16 columns per 128 rows of H (256 columns
// at H = 2048).  All waits are bounded mbarrier waits; a failed wait raises the error flag, every
// role leaves its loops, the producer waits for copies in flight and TMEM is freed.
#include <cuda.h>

#include <cstring>

#include "remoe_internal.cuh"
#include "tma_ring.cuh"
#include "batched_plan.cuh"

namespace remoe {

namespace {

constexpr int kTcTokTile = 16;
constexpr int kTcBlockCh = 64;
constexpr int kTcThreads = 192;
constexpr int kTileBytes = 16384;                      // one operand tile: 128 rows x 128 B
constexpr int kStageTiles = 2;                         // tiles per ring stage (one bulk copy, one barrier round trip)
constexpr int kStageBytes = kStageTiles * kTileBytes;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kD2Col = 32;                        // D1 buffers at columns 0 and 16, D2 tiles from column 32

using namespace ring;

__device__ __forceinline__ void tma_load_3d(void* dst, const CUtensorMap* map, int c0, int c1, int c2, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          smem_u32(dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}
// Shared-memory matrix descriptor, 128-byte swizzle: start address, leading and stride byte
// offsets in 16-byte units, descriptor version 1 in bits 46-47, layout type 2 in bits 61-63.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr >> 4) & 0x3fffu) | ((uint64_t)((lbo_bytes >> 4) & 0x3fffu) << 16) |
         ((uint64_t)((sbo_bytes >> 4) & 0x3fffu) << 32) | ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// Instruction descriptor: fp32 accumulate (bits 4-5 = 1), bf16 A and B (bits 7-9, 10-12 = 1),
// N >> 3 in bits 17-22, M >> 4 in bits 24-28; bit 15 set = A is MN-major.
constexpr uint32_t kIdescK = (1u << 4) | (1u << 7) | (1u << 10) | ((kTcTokTile >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescMN = kIdescK | (1u << 15);

__device__ __forceinline__ void umma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}" ::"r"(tmem_d),
      "l"(da), "l"(db), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// Arrives on `bar` once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
// 16 consecutive fp32 columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}
// The same load without the wait: the caller issues several, then one tcgen05.wait::ld, and only
// then reads the values.
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t taddr, float* v) {
  uint32_t* r = reinterpret_cast<uint32_t*>(v);
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

// Tensor maps over the staging pool (channel-major blocks as fetched), viewed as [H, 3, channel rows]:
// box {64, 2, 64} = gate/up rows of 64 channels x 64 columns, box {64, 1, 64} = W_down rows.
struct TcMaps {
  CUtensorMap stage_gu, stage_d;
};

// Walks the 64-channel groups of a CTA's unit range in order, piece by piece.
struct GroupRec {
  PieceInfo p;
  int blk;          // channel block within the expert
  int np;           // running piece number within this CTA
  int idx;          // running group number within this CTA
  bool first, last; // first / last group of its piece
};
struct GroupWalk {
  const BatchArgs& a;
  int n_items, ua, ub, j, np, idx, blk;
  PieceInfo p;
  bool in_piece;
  __device__ GroupWalk(const BatchArgs& a_, int n_items_, int ua_, int ub_, int j0)
      : a(a_), n_items(n_items_), ua(ua_), ub(ub_), j(j0), np(-1), idx(0), blk(0), in_piece(false) {}
  __device__ bool next(GroupRec& g) {
    while (!in_piece) {
      if (j >= n_items || a.plan[kPlanHeader + 4 * j + 3] >= ub) return false;
      const bool got = make_piece(a, j, ua, ub, p);
      ++j;
      if (got && p.blk0 < p.blk1) { in_piece = true; blk = p.blk0; ++np; }
    }
    g.p = p; g.blk = blk; g.np = np; g.idx = idx++;
    g.first = blk == p.blk0;
    g.last = blk + 1 == p.blk1;
    if (++blk == p.blk1) in_piece = false;
    return true;
  }
};

template <int H>
struct TcGeo {
  static constexpr int kChunks = H / 64;               // K chunks of the first contraction
  static constexpr int kTiles = H / 128;               // output tiles of the second contraction
  static constexpr int kB1Bytes = kChunks * 2048;      // X^T: 16 tokens x 128 B per chunk
  static constexpr int kB2Bytes = 2048;                // a: 16 tokens x 64 channels
  static constexpr int kFixed = kB1Bytes + kB2Bytes;
  static constexpr int kStages = (227 * 1024 - 2048 - kFixed) / kStageBytes > 5 ? 5 : (227 * 1024 - 2048 - kFixed) / kStageBytes;
  static constexpr size_t kSmem = 1024 + kFixed + (size_t)kStages * kStageBytes + 512;
  static_assert(kChunks % kStageTiles == 0 && kTiles % kStageTiles == 0, "a stage never spans two tile kinds");
};

template <int H>
__global__ void __launch_bounds__(kTcThreads, 1)
ffn_batched_tc_kernel(const __grid_constant__ BatchArgs a) {
  using G = TcGeo<H>;
  constexpr int NS = G::kStages;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* b1 = smem;
  unsigned char* b2 = b1 + G::kB1Bytes;
  unsigned char* ring = b2 + G::kB2Bytes;                              // 1024-byte aligned
  uint64_t* bars = reinterpret_cast<uint64_t*>(ring + (size_t)NS * kStageBytes);
  uint64_t *full = bars, *empty = bars + NS;
  uint64_t* x_full = bars + 2 * NS;        // X^T of a piece staged            (128 epilogue threads)
  uint64_t* x_empty = x_full + 1;          // X^T no longer read                 (commit)
  uint64_t* d1_full = x_full + 2;          // [2] first contraction of a group done (commit)
  uint64_t* d1_empty = x_full + 4;         // [2] D1 buffer read out             (128 threads)
  uint64_t* b2_full = x_full + 6;          // activations of a group staged      (128 threads)
  uint64_t* b2_empty = x_full + 7;         // second contraction of a group done (commit)
  uint64_t* d2_full = x_full + 8;          // a piece's output complete          (commit)
  uint64_t* d2_empty = x_full + 9;         // a piece's output read out          (128 threads)
  uint64_t* drain = x_full + 10;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(x_full + 11);
  __shared__ int s_abort;

  const DevStack& d = a.d;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int BK = d.B * d.K, P = d.K + d.S;

  if (tid == 0) {
    s_abort = 0;
    for (int s = 0; s < NS; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
    mbar_init(x_full, 128); mbar_init(x_empty, 1);
    mbar_init(d1_full, 1); mbar_init(d1_full + 1, 1);
    mbar_init(d1_empty, 128); mbar_init(d1_empty + 1, 128);
    mbar_init(b2_full, 128); mbar_init(b2_empty, 1);
    mbar_init(d2_full, 1); mbar_init(d2_empty, 128);
    mbar_init(drain, 1);
    mbar_fence_init();
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  const int n_items = a.plan[0], n_units = a.plan[1];
  const int q = (n_units + (int)gridDim.x - 1) / (int)gridDim.x;
  const int ua = min(n_units, (int)blockIdx.x * q), ub = min(n_units, ua + q);
  const bool have_work = ua < ub;
  const int j0 = have_work ? first_item(a, n_items, ua) : 0;
  auto aborted = [&]() { return *(volatile int*)&s_abort != 0; };
  auto fail = [&](int code) { atomicCAS(d.err, kErrNone, code); atomicExch(&s_abort, 1); };

  if (have_work && warp == 4) {
    // ---------------------------------------------------------------- TMA producer
    // Tile order: A1(g0); A1(g1), A2(g0); A1(g2), A2(g1); ... ; A2(last) -- the order the MMA
    // thread consumes them in.
    if (lane == 0) {
      int n = 0;
      bool ok = true;
      auto emit = [&](const GroupRec& g, bool second) {
        // tiles of this group in the block: A1 tiles first, then the A2 tiles
        const char* src = g.p.base + ((size_t)g.blk * (G::kChunks + G::kTiles) + (second ? G::kChunks : 0)) * kTileBytes;
        const int stages = (second ? G::kTiles : G::kChunks) / kStageTiles;
        for (int t = 0; t < stages && ok; ++t, ++n) {
          const int s = n % NS;
          if (n >= NS && (aborted() || !mbar_wait(empty + s, ((n / NS) - 1) & 1))) {
            if (!aborted()) fail(kErrWaitEmpty);
            ok = false;
            break;
          }
          mbar_expect_tx(full + s, kStageBytes);
          bulk_g2s(ring + (size_t)s * kStageBytes, src + (size_t)t * kStageBytes, kStageBytes, full + s);
        }
      };
      GroupWalk walk(a, n_items, ua, ub, j0);
      GroupRec g, prev;
      bool have_prev = false;
      while (ok && walk.next(g)) {
        emit(g, false);
        if (have_prev && ok) emit(prev, true);
        prev = g;
        have_prev = true;
      }
      if (have_prev && ok) emit(prev, true);
      if (!ok) {
        for (int m = max(0, n - NS); m < n; ++m)
          if (!mbar_wait(full + (m % NS), (m / NS) & 1)) atomicCAS(d.err, kErrNone, kErrDrain);
      }
    }
  } else if (have_work && warp == 5) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      int n = 0;
      bool ok = true;
      // first contraction of a group into D1 buffer (idx & 1)
      auto gemm1 = [&](const GroupRec& g) {
        if (g.first) ok = !aborted() && mbar_wait(x_full, g.np & 1);
        if (ok && g.idx >= 2) ok = !aborted() && mbar_wait(d1_empty + (g.idx & 1), ((g.idx >> 1) - 1) & 1);
        const uint32_t dcol = tmem + (uint32_t)(g.idx & 1) * 16;
        for (int kc = 0; kc < G::kChunks && ok; kc += kStageTiles, ++n) {
          const int s = n % NS;
          ok = !aborted() && mbar_wait(full + s, (n / NS) & 1);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int j = 0; j < kStageTiles; ++j) {
            const uint32_t a_addr = smem_u32(ring + (size_t)s * kStageBytes + j * kTileBytes);
            const uint32_t b_addr = smem_u32(b1 + (kc + j) * 2048);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma(dcol, smem_desc(a_addr + k * 32, 16, 1024), smem_desc(b_addr + k * 32, 16, 1024), kIdescK,
                   (kc | j | k) ? 1u : 0u);
          }
          umma_commit(empty + s);
        }
        if (!ok) return;
        umma_commit(d1_full + (g.idx & 1));
        if (g.last) umma_commit(x_empty);                          // X^T of this piece is no longer needed
      };
      // second contraction of a group into the piece's output tiles
      auto gemm2 = [&](const GroupRec& g) {
        ok = !aborted() && mbar_wait(b2_full, g.idx & 1);
        if (ok && g.first && g.np > 0) ok = !aborted() && mbar_wait(d2_empty, (g.np - 1) & 1);
        tc_fence_after();
        for (int ht = 0; ht < G::kTiles && ok; ht += kStageTiles, ++n) {
          const int s = n % NS;
          ok = !aborted() && mbar_wait(full + s, (n / NS) & 1);
          if (!ok) break;
          tc_fence_after();
          const uint32_t b_addr = smem_u32(b2);
#pragma unroll
          for (int j = 0; j < kStageTiles; ++j) {
            const uint32_t a_addr = smem_u32(ring + (size_t)s * kStageBytes + j * kTileBytes);
#pragma unroll
            for (int k = 0; k < 4; ++k)
              umma(tmem + kD2Col + (ht + j) * 16, smem_desc(a_addr + k * 2048, 8192, 1024),
                   smem_desc(b_addr + k * 32, 16, 1024), kIdescMN, (!g.first || k) ? 1u : 0u);
          }
          umma_commit(empty + s);
        }
        if (!ok) return;
        umma_commit(b2_empty);
        if (g.last) umma_commit(d2_full);
      };
      GroupWalk walk(a, n_items, ua, ub, j0);
      GroupRec g, prev;
      bool have_prev = false;
      while (ok && walk.next(g)) {
        gemm1(g);
        if (have_prev && ok) gemm2(prev);
        prev = g;
        have_prev = true;
      }
      if (have_prev && ok) gemm2(prev);
      if (!ok) {
        if (!aborted()) fail(kErrWaitFull);
        umma_commit(drain);                                       // let the tensor cores finish before TMEM is freed
        mbar_wait(drain, 0);
      }
    }
  } else if (have_work) {
    // ------------------------------------------------------------- epilogue warps 0-3
    bool ok = true;
    const uint32_t lane_base = (uint32_t)(warp * 32) << 16;
    auto tok_of = [&](const PieceInfo& p, int t) -> int {
      if (t >= p.n_tok) return -1;
      return p.shared ? p.tile * kTcTokTile + t : d.grp_tok[(p.l * BK + p.cand) * d.B + p.tile * kTcTokTile + t];
    };
    auto kq_of = [&](const PieceInfo& p, int t) -> int {
      return p.shared ? d.K + (p.cand - BK) : d.grp_k[(p.l * BK + p.cand) * d.B + p.tile * kTcTokTile + t];
    };
    // X^T tile of a piece: 16 tokens x H as bf16, 128-byte rows per 64-column chunk, 16-byte pieces
    // XORed with the row number (the 128-byte swizzle the MMA descriptors expect).
    auto stage_x = [&](const PieceInfo& p) {
      constexpr int kPer = (H / 8 + 127) / 128;         // 16-byte pieces per thread and token
#pragma unroll 2
      for (int t = 0; t < kTcTokTile; ++t) {
        const int tok = tok_of(p, t);
        float4 x[kPer][2];
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          x[i][0] = x[i][1] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (tok >= 0 && tid + 128 * i < H / 8) {
            const float4* src =
                reinterpret_cast<const float4*>(a.hidden_in + ((size_t)p.l * d.B + tok) * H + (tid + 128 * i) * 8);
            x[i][0] = __ldg(src);
            x[i][1] = __ldg(src + 1);
          }
        }
#pragma unroll
        for (int i = 0; i < kPer; ++i) {
          const int c8 = tid + 128 * i, kc = c8 >> 3, c = c8 & 7;
          if (c8 < H / 8)
            *reinterpret_cast<uint4*>(b1 + kc * 2048 + t * 128 + ((c ^ (t & 7)) << 4)) =
              make_uint4(pack_bf16(x[i][0].x, x[i][0].y), pack_bf16(x[i][0].z, x[i][0].w),
                         pack_bf16(x[i][1].x, x[i][1].y), pack_bf16(x[i][1].z, x[i][1].w));
        }
      }
      proxy_fence();
      mbar_arrive(x_full);
    };
    float sc[kTcTokTile];
    auto load_scales = [&](const PieceInfo& p) {
#pragma unroll
      for (int t = 0; t < kTcTokTile; ++t) {
        const int tok = tok_of(p, t);
        sc[t] = tok < 0 ? 0.f
                        : (p.shared ? d.shared_scale[p.l * d.B + tok]
                                    : a.gates[((size_t)p.l * d.B + tok) * d.K + kq_of(p, t)]);
      }
    };
    // piece done: read the output tiles and write one stamped partial row per (token, rank)
    auto read_out = [&](const GroupRec& g) {
      ok = !aborted() && mbar_wait(d2_full, g.np & 1);
      if (!ok) return;
      tc_fence_after();
      size_t rows[kTcTokTile];
#pragma unroll
      for (int t = 0; t < kTcTokTile; ++t) {
        const int tok = tok_of(g.p, t);
        rows[t] = tok < 0 ? (size_t)-1
                          : (((size_t)g.p.l * d.B + tok) * P + kq_of(g.p, t)) * kUnitsPerItem + g.p.first_unit;
      }
      constexpr int kBatch = G::kTiles >= 4 ? 4 : G::kTiles;
      for (int ht0 = 0; ht0 < G::kTiles; ht0 += kBatch) {
        float v[kBatch][16];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) tmem_ld16_nowait(tmem + lane_base + kD2Col + (ht0 + i) * 16, v[i]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
          const int h = (ht0 + i) * 128 + warp * 32 + lane;
#pragma unroll
          for (int t = 0; t < kTcTokTile; ++t)
            if (rows[t] != (size_t)-1) a.part[rows[t] * H + h] = v[i][t];
        }
      }
      tc_fence_before();
      mbar_arrive(d2_empty);
#pragma unroll
      for (int t = 0; t < kTcTokTile; ++t)
        if (tid == t && rows[t] != (size_t)-1) a.flags[rows[t]] = a.step_id;
    };

    GroupWalk walk(a, n_items, ua, ub, j0);
    GroupRec g, gn;
    bool have = walk.next(g);
    if (have) stage_x(g.p);
    while (have && ok) {
      if (g.first) load_scales(g.p);
      // activation step of group g: D1 buffer (idx & 1) -> a -> second B operand
      ok = !aborted() && mbar_wait(d1_full + (g.idx & 1), (g.idx >> 1) & 1);
      if (!ok) break;
      tc_fence_after();
      float v[16];
      tmem_ld16(tmem + lane_base + (uint32_t)(g.idx & 1) * 16, v);
      tc_fence_before();
      mbar_arrive(d1_empty + (g.idx & 1));
      if (g.idx > 0) ok = !aborted() && mbar_wait(b2_empty, (g.idx - 1) & 1);
      if (!ok) break;
      const int ch = (warp * 32 + lane) >> 1;       // lane 2c holds the gate row of channel c, lane 2c+1 its up row
#pragma unroll
      for (int t = 0; t < kTcTokTile; ++t) {
        const float u = __shfl_down_sync(kFull, v[t], 1);
        if ((lane & 1) == 0) {
          const float av = v[t] / (1.f + __expf(-v[t])) * u * sc[t];
          *reinterpret_cast<unsigned short*>(b2 + t * 128 + (((ch >> 3) ^ (t & 7)) << 4) + ((ch & 7) << 1)) =
              (unsigned short)(pack_bf16(av, 0.f) & 0xffffu);
        }
      }
      proxy_fence();
      mbar_arrive(b2_full);

      const bool have_next = walk.next(gn);
      if (g.last) {
        if (have_next) {
          // the next piece's X^T may replace this one's as soon as its last first-contraction is done
          ok = !aborted() && mbar_wait(x_empty, g.np & 1);
          if (!ok) break;
          stage_x(gn.p);
        }
        read_out(g);
      }
      have = have_next;
      g = gn;
    }
    if (!ok && !aborted()) fail(kErrWaitFull);
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 0)
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// ------------------------------------------------------------------------------------ retile
// Channel-major block (as fetched from the host) -> operand-tile order.  One CTA per (64-channel
// group, block): its 48 tiles (H = 2048) are loaded through the staging pool's tensor maps into a
// small ring, swizzled by the TMA unit, and written out as contiguous 16 KB runs with bulk stores.
constexpr int kRetileStages = 6;
constexpr int kRetileJobs = 64;
struct RetileArgs {
  int n, inter;                     // jobs in this launch; intermediate size of the blocks
  int src_row[kRetileJobs];         // first channel row of the block within the staging pool
  char* dst[kRetileJobs];           // destination block (slot or shared block)
  int* err;
};
__device__ __forceinline__ void bulk_s2g(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(__cvta_generic_to_global(dst)),
               "r"(smem_u32(src)), "r"(bytes)
               : "memory");
}

template <int H>
__global__ void __launch_bounds__(32) retile_kernel(const __grid_constant__ TcMaps maps,
                                                    const __grid_constant__ RetileArgs r) {
  using G = TcGeo<H>;
  constexpr int NS = kRetileStages, T = G::kChunks + G::kTiles;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* ring = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint64_t* full = reinterpret_cast<uint64_t*>(ring + (size_t)NS * kTileBytes);
  if (threadIdx.x != 0) return;
  for (int s = 0; s < NS; ++s) mbar_init(full + s, 1);
  mbar_fence_init();
  const int row = r.src_row[blockIdx.y] + (int)blockIdx.x * kTcBlockCh;
  char* dst = r.dst[blockIdx.y] + (size_t)blockIdx.x * T * kTileBytes;
  auto issue = [&](int t) {
    const int s = t % NS;
    unsigned char* st = ring + (size_t)s * kTileBytes;
    mbar_expect_tx(full + s, kTileBytes);
    if (t < G::kChunks) {
      tma_load_3d(st, &maps.stage_gu, t * 64, 0, row, full + s);
    } else {
      const int ht = t - G::kChunks;
      tma_load_3d(st, &maps.stage_d, ht * 128, 2, row, full + s);
      tma_load_3d(st + kTileBytes / 2, &maps.stage_d, ht * 128 + 64, 2, row, full + s);
    }
  };
  int issued = 0;
  for (; issued < NS && issued < T; ++issued) issue(issued);
  bool ok = true;
  for (int t = 0; t < T; ++t) {
    const int s = t % NS;
    if (!mbar_wait(full + s, (t / NS) & 1)) { ok = false; break; }
    proxy_fence();
    bulk_s2g(dst + (size_t)t * kTileBytes, ring + (size_t)s * kTileBytes, kTileBytes);
    asm volatile("cp.async.bulk.commit_group;" ::: "memory");
    if (issued < T) {
      asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");     // the stage has been read out
      issue(issued++);
    }
  }
  asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  if (!ok) {
    atomicCAS(r.err, kErrNone, kErrWaitFull);
    // loads still in flight must land before the CTA's shared memory is given up
    for (int t = max(0, issued - NS); t < issued; ++t)
      if (!mbar_wait(full + (t % NS), (t / NS) & 1)) atomicCAS(r.err, kErrNone, kErrDrain);
  }
}

// ------------------------------------------------------------------- low-precision widen + retile
// A batched stack over an FP8 E4M3 (value = byte * 2^-8) or a 4-bit grouped host store fetches the stored bytes
// -- a half or 0.28 of what a bf16 block moves over the host link -- and keeps its slots as bf16 operand tiles,
// so the MMA kernel above is the same.  This kernel does both steps at once for freshly fetched channel-major
// blocks: every 16-byte piece of an operand tile is eight consecutive stored elements of one row, widened to
// bf16 and written at the swizzled place the tensor-map path would have put it.  FP8 widens exactly (an E4M3
// value times 2^-8 has at most 4 significant bits); a 4-bit value (code - 8) * bf16 scale has up to 11 and is
// rounded to nearest even once.  One CTA per (64-channel group, block); plain loads and stores.
struct WidenArgs {
  int n, inter;
  const unsigned char* src[kRetileJobs];   // channel-major stored block in the staging pool
  char* dst[kRetileJobs];                  // destination block (slot or shared block), bf16 tile order
};

// WB: 1 = FP8 E4M3 bytes, 0 = 4-bit grouped format
template <int H, int WB>
__global__ void __launch_bounds__(256) widen_retile_kernel(const __grid_constant__ WidenArgs r) {
  using G = TcGeo<H>;
  constexpr int T = G::kChunks + G::kTiles;
  constexpr size_t kRow = weight_row_bytes(H, WB);
  const unsigned char* src = r.src[blockIdx.y] + (size_t)blockIdx.x * kTcBlockCh * 3 * kRow;
  char* dst = r.dst[blockIdx.y] + (size_t)blockIdx.x * T * kTileBytes;
  for (int q = threadIdx.x; q < T * 1024; q += 256) {
    const int t = q >> 10, line = (q >> 3) & 127, pos = q & 7;
    const int c = pos ^ (line & 7);                      // which 8 columns of the line sit at this place
    int ch, kind, col;
    if (t < G::kChunks) {                                // A1 tile: lines alternate gate / up of a channel
      ch = line >> 1; kind = line & 1; col = t * 64 + c * 8;
    } else {                                             // A2 tile: two halves of 64 channel lines
      ch = line & 63; kind = 2; col = (t - G::kChunks) * 128 + (line >> 6) * 64 + c * 8;
    }
    const unsigned char* row = src + ((size_t)ch * 3 + kind) * kRow;
    float f[8];
    if constexpr (WB == 1) {
      const uint2 b = __ldg(reinterpret_cast<const uint2*>(row + col));
      Elems<1>::pair(b.x & 0xffffu, f[0], f[1]); Elems<1>::pair(b.x >> 16, f[2], f[3]);
      Elems<1>::pair(b.y & 0xffffu, f[4], f[5]); Elems<1>::pair(b.y >> 16, f[6], f[7]);
      constexpr float k = WScale<1>::kDot;               // the store's power-of-two scale
#pragma unroll
      for (int i = 0; i < 8; ++i) f[i] *= k;
    } else {
      const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(row + col / 2));        // eight codes
      const float sc = __uint_as_float(
          (uint32_t)__ldg(reinterpret_cast<const unsigned short*>(row + H / 2 + 2 * (col / 32))) << 16);
#pragma unroll
      for (int i = 0; i < 8; ++i) f[i] = (float)((int)((w >> (4 * i)) & 0xfu) - 8) * sc;
    }
    *reinterpret_cast<uint4*>(dst + (size_t)t * kTileBytes + line * 128 + pos * 16) =
        make_uint4(pack_bf16(f[0], f[1]), pack_bf16(f[2], f[3]), pack_bf16(f[4], f[5]), pack_bf16(f[6], f[7]));
  }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// A pool of channel-major expert blocks as a 3-D bf16 tensor (H columns, 3 row kinds, channel rows).
bool encode_pool(EncodeTiledFn encode, CUtensorMap* gu, CUtensorMap* dn, const void* base, int H, size_t rows) {
  cuuint64_t dims[3] = {(cuuint64_t)H, 3, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)H * 2, (cuuint64_t)3 * H * 2};
  cuuint32_t box_gu[3] = {64, 2, 64}, box_d[3] = {64, 1, 64}, estr[3] = {1, 1, 1};
  void* p = const_cast<void*>(base);
  return encode(gu, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, p, dims, strides, box_gu, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS &&
         encode(dn, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, p, dims, strides, box_d, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int H>
cudaError_t launch_tc(const BatchArgs& a, int grid, cudaStream_t st) {
  static std::atomic<bool> configured[kMaxDevices];
  cudaError_t e = allow_dynamic_smem(ffn_batched_tc_kernel<H>, TcGeo<H>::kSmem, configured);
  if (e != cudaSuccess) return e;
  BatchArgs b = a;
  b.tok_tile = kTcTokTile;
  b.blk_ch = kTcBlockCh;
  plan_kernel<<<1, 1024, 0, st>>>(b);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  ffn_batched_tc_kernel<H><<<grid, kTcThreads, TcGeo<H>::kSmem, st>>>(b);
  return cudaGetLastError();
}

template <int H>
cudaError_t launch_retile(const TcMaps& maps, const RetileArgs& r, cudaStream_t st) {
  constexpr size_t kSmem = 1024 + (size_t)kRetileStages * kTileBytes + 64;
  static std::atomic<bool> configured[kMaxDevices];
  cudaError_t e = allow_dynamic_smem(retile_kernel<H>, kSmem, configured);
  if (e != cudaSuccess) return e;
  retile_kernel<H><<<dim3(r.inter / kTcBlockCh, r.n), 32, kSmem, st>>>(maps, r);
  return cudaGetLastError();
}

}  // namespace

bool ffn_batched_tc_supported(const DevStack& d) {
  if (d.wbytes != 2) return false;
  if (d.H != 256 && d.H != 512 && d.H != 1024 && d.H != 2048) return false;
  if (d.I % kTcBlockCh || (d.S && d.Is % kTcBlockCh)) return false;
  return true;
}

size_t ffn_batched_tc_maps_bytes() { return sizeof(TcMaps); }

cudaError_t ffn_batched_tc_init(const DevStack& d, const void* stage_pool, size_t stage_bytes, void* maps_out) {
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (!fn) return cudaErrorNotSupported;
  TcMaps* m = static_cast<TcMaps*>(maps_out);
  const size_t rows = stage_bytes / ((size_t)3 * d.H * 2);
  if (rows < (size_t)kTcBlockCh || rows > 0x7fffffffu) return cudaErrorInvalidValue;
  if (!encode_pool(reinterpret_cast<EncodeTiledFn>(fn), &m->stage_gu, &m->stage_d, stage_pool, d.H, rows))
    return cudaErrorInvalidValue;
  return cudaSuccess;
}

cudaError_t launch_ffn_batched_tc(const BatchArgs& a, int grid, cudaStream_t st) {
  switch (a.d.H) {
    case 256: return launch_tc<256>(a, grid, st);
    case 512: return launch_tc<512>(a, grid, st);
    case 1024: return launch_tc<1024>(a, grid, st);
    case 2048: return launch_tc<2048>(a, grid, st);
  }
  return cudaErrorInvalidValue;
}

template <int WB>
cudaError_t launch_widen(const DevStack& d, const WidenArgs& r, dim3 grid, cudaStream_t st) {
  switch (d.H) {
    case 256: widen_retile_kernel<256, WB><<<grid, 256, 0, st>>>(r); break;
    case 512: widen_retile_kernel<512, WB><<<grid, 256, 0, st>>>(r); break;
    case 1024: widen_retile_kernel<1024, WB><<<grid, 256, 0, st>>>(r); break;
    case 2048: widen_retile_kernel<2048, WB><<<grid, 256, 0, st>>>(r); break;
    default: return cudaErrorInvalidValue;
  }
  return cudaGetLastError();
}

cudaError_t launch_widen_retile_tc(const DevStack& d, int src_wbytes, int n, const void* const* src, char* const* dst,
                                   int inter, cudaStream_t st) {
  if (src_wbytes != 0 && src_wbytes != 1) return cudaErrorInvalidValue;
  for (int i0 = 0; i0 < n; i0 += kRetileJobs) {
    WidenArgs r{};
    r.n = n - i0 < kRetileJobs ? n - i0 : kRetileJobs;
    r.inter = inter;
    for (int i = 0; i < r.n; ++i) {
      if (reinterpret_cast<uintptr_t>(src[i0 + i]) & 7u) return cudaErrorInvalidValue;
      r.src[i] = static_cast<const unsigned char*>(src[i0 + i]);
      r.dst[i] = dst[i0 + i];
    }
    const dim3 grid(inter / kTcBlockCh, r.n);
    const cudaError_t e = src_wbytes == 1 ? launch_widen<1>(d, r, grid, st) : launch_widen<0>(d, r, grid, st);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_retile_tc(const DevStack& d, const void* maps, int n, const size_t* src_offsets,
                             char* const* dst, int inter, cudaStream_t st) {
  const TcMaps& m = *static_cast<const TcMaps*>(maps);
  const size_t row_bytes = (size_t)3 * d.H * 2;
  for (int i0 = 0; i0 < n; i0 += kRetileJobs) {
    RetileArgs r{};
    r.n = n - i0 < kRetileJobs ? n - i0 : kRetileJobs;
    r.inter = inter;
    r.err = d.err;
    for (int i = 0; i < r.n; ++i) {
      if (src_offsets[i0 + i] % row_bytes) return cudaErrorInvalidValue;
      r.src_row[i] = (int)(src_offsets[i0 + i] / row_bytes);
      r.dst[i] = dst[i0 + i];
    }
    cudaError_t e = cudaErrorInvalidValue;
    switch (d.H) {
      case 256: e = launch_retile<256>(m, r, st); break;
      case 512: e = launch_retile<512>(m, r, st); break;
      case 1024: e = launch_retile<1024>(m, r, st); break;
      case 2048: e = launch_retile<2048>(m, r, st); break;
    }
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

}  // namespace remoe

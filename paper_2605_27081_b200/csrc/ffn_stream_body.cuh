// The per-CTA body of the expert-streaming GEMV, shared by the stack kernel (ffn_stream.cu) and the
// allocation-free single-layer entry point (ffn_static.cu).
//
// A launch streams a list of weight rows.  A row is one channel triple of an expert block, W_gate[i,:],
// W_up[i,:], W_down[:,i], contiguous in memory; the list is the concatenation of the blocks of the launch's
// (layer, expert) pairs, described by an exclusive prefix table of rows per pair.  One CTA owns the
// contiguous range [r0, r1) of that list:
//   - kProducerLanes lanes of the producer warp bring rows into a ring of shared-memory stages with bulk
//     asynchronous copies (one row per stage), guarded by full / empty mbarriers;
//   - kConsumerWarps warps take rows round-robin; a warp owns a whole row triple: two dot products with h by
//     16-byte shared loads and a shuffle reduction, SiLU, then an AXPY of the third row into the warp's
//     private fp32 copy of out[H] held in registers;
//   - at every layer boundary, and at the end, the private copies are added in warp order and written as this
//     CTA's partial for that layer.
// Where the rows come from and where the partials go is the caller's business, passed as a `Work` object:
//   const char* base(int pair, bool& ok)   first row of the pair's block (ok = false: bad index, give up)
//   float scale(int pair, int layer)       gate weight / shared-expert scale of the pair
//   const float* hidden(int layer)         h of the layer, [H] float32
//   float* partial(int layer)              where this CTA's partial of the layer goes, [H] float32
//   void fail(int code)                    record a device-side error code
//   static constexpr bool kPoison          on a wait that ran out, fill the partial with NaN (no error word)
// Every wait is bounded by `spin` polls; when one runs out the role records the error, all roles leave their
// loops, and the producer lanes wait (bounded again) for the copies they still have in flight.
#pragma once

#include "remoe_internal.cuh"
#include "tma_ring.cuh"

namespace remoe {
namespace stream {

constexpr int kConsumerWarps = 8;
constexpr int kThreads = (kConsumerWarps + 1) * 32;
constexpr int kMaxStages = 16;                 // multiple of kConsumerWarps
constexpr int kProducerLanes = 4;              // divides kConsumerWarps, hence every ring depth

// The ring depth is a multiple of the consumer-warp count, so a stage is always consumed by the same
// warp.  That warp has waited for fill k-1 of the stage before it waits for fill k, hence the barrier can
// never be a whole phase behind the parity it is asked about (a parity wait cannot tell "phase k done"
// from "phase k-2 done").
struct Ring {
  uint64_t* full;
  uint64_t* empty;
  float* red;                  // [kConsumerWarps][32 * kVec] exchange buffer of the layer flush
  unsigned char* stages;       // [n_stages][3 rows]
  int n_stages;
  int* abort_flag;             // shared-memory word: some role gave up
};

template <int WB, int H, class Work>
__device__ __forceinline__ void stream_rows(const Work& wk, const int* prefix, int P, int r0, int r1, const Ring& ring,
                                            unsigned spin, int lose_row1) {
  using namespace remoe::ring;
  using E = Elems<WB>;
  constexpr int kVec = E::kVec;
  constexpr int kIter = H / (32 * kVec);
  constexpr int kCols = kIter * kVec;                  // columns of h / out owned by one lane
  constexpr uint32_t kRowBytes = (uint32_t)weight_row_bytes(H, WB);
  constexpr uint32_t kStageBytes = 3u * kRowBytes;
  constexpr bool kGrouped = WB == 0;                   // per-group scales follow the codes of a row

  uint64_t* full = ring.full;
  uint64_t* empty = ring.empty;
  unsigned char* stages = ring.stages;
  const int NS = ring.n_stages;
  volatile int* s_abort = ring.abort_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

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
          base = wk.base(pair, ok);
          if (!ok) break;
          pair_of_base = pair;
        }
        const int i = r - prefix[pair];
        const int n = r - r0, s = n % NS;
        if (n >= NS) {
          if (*s_abort) { ok = false; break; }
          if (!mbar_wait(empty + s, ((n / NS) - 1) & 1, spin)) {
            wk.fail(kErrWaitEmpty);
            ok = false;
            break;
          }
        }
        if (r + 1 == lose_row1) continue;              // test aid: this stage is never filled
        mbar_expect_tx(full + s, kStageBytes);
        bulk_g2s(stages + (size_t)s * kStageBytes, base + (size_t)i * kStageBytes, kStageBytes, full + s);
      }
      if (!ok || *s_abort) {
        // Let the consumers leave, then wait (bounded) for copies that are still landing.
        atomicExch(ring.abort_flag, 1);
        for (int n = issued - kProducerLanes; n >= 0 && n >= issued - NS; n -= kProducerLanes)
          if (!mbar_wait(full + (n % NS), (n / NS) & 1, spin)) wk.fail(kErrDrain);
      }
    }
    return;
  }

  // ----------------------------------------------------------------- consumers
  float hreg[kCols], acc[kCols];
  int pair = 0;
  while (prefix[pair + 1] <= r0) ++pair;
  const int l_first = pair / P;
  int pair_last = pair;
  while (prefix[pair_last + 1] < r1) ++pair_last;
  const int l_last = pair_last / P;
  bool aborted = false;

  for (int l = l_first; l <= l_last; ++l) {
    const int lo = max(r0, prefix[l * P]), hi = min(r1, prefix[(l + 1) * P]);
    if (lo >= hi) continue;
    const float* h = wk.hidden(l);
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
    // grouped format: the decoded codes carry an offset that is taken out once per group -- from a dot product
    // with the sum of this lane's h over the group, from the AXPY with the sum of the row activations
    float hsum[kGrouped ? kIter : 1], asum[kGrouped ? kIter : 1];
    if constexpr (kGrouped) {
#pragma unroll
      for (int it = 0; it < kIter; ++it) {
        float t = 0.f;
#pragma unroll
        for (int j = 0; j < kVec; ++j) t += hreg[it * kVec + j];
        hsum[it] = t * E::kBias;
        asum[it] = 0.f;
      }
    }

    // first row of this layer handled by this warp: local index n = r - r0 with n % 8 == warp
    int r = lo + ((warp - (lo - r0)) % kConsumerWarps + kConsumerWarps) % kConsumerWarps;
    float scale = 0.f;
    int pair_of_scale = -1;
    for (; r < hi && !aborted; r += kConsumerWarps) {
      while (prefix[pair + 1] <= r) ++pair;
      if (pair != pair_of_scale) {
        scale = wk.scale(pair, l);
        pair_of_scale = pair;
      }
      const int n = r - r0, s = n % NS;
      // decided for the whole warp: the shuffles below need every lane
      if (__any_sync(kFull, *s_abort || !mbar_wait(full + s, (n / NS) & 1, spin))) {
        if (!*s_abort) { wk.fail(kErrWaitFull); atomicExch(ring.abort_flag, 1); }
        aborted = true;
        if (Work::kPoison) {
#pragma unroll
          for (int c = 0; c < kCols; ++c) acc[c] = __int_as_float(0x7fc00000);
        }
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
          g = fmaf(E::scale(st, H, it * 32 + lane), t - hsum[it], g);
        }
#pragma unroll
        for (int it = 0; it < kIter; ++it) {
          float w[kVec], t = 0.f;
          E::load(st + kRowBytes + (it * 32 + lane) * 16, w);
#pragma unroll
          for (int j = 0; j < kVec; ++j) t = fmaf(w[j], hreg[it * kVec + j], t);
          u = fmaf(E::scale(st + kRowBytes, H, it * 32 + lane), t - hsum[it], u);
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
        if constexpr (kGrouped) asum[it] += a_it;
#pragma unroll
        for (int j = 0; j < kVec; ++j) acc[it * kVec + j] = fmaf(a_it, w[j], acc[it * kVec + j]);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(empty + s);
    }

    if constexpr (kGrouped) {
#pragma unroll
      for (int it = 0; it < kIter; ++it)
#pragma unroll
        for (int j = 0; j < kVec; ++j) acc[it * kVec + j] = fmaf(-E::kBias, asum[it], acc[it * kVec + j]);
    }
    // Layer flush: add the eight private copies in warp order, write this CTA's partial.
    // One pass per 32*kVec columns keeps the exchange buffer at a few KB.
    float* dst = wk.partial(l);
    float* red = ring.red;
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

}  // namespace stream
}  // namespace remoe

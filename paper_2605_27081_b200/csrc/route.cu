// Router GEMV, softmax, top-K gating, reuse statistic and cache directory update.
//
// One CTA per (layer, sequence) computes the N router logits (Sec. 3.1: h^T theta_gate) with
// one warp per expert row, 128-bit loads and shuffle reductions.  Warp 0 then takes the
// softmax over all N logits, selects the K largest logits (equal logits: lower index first),
// emits ids and gate weights, and updates the reuse statistic |E_t n E_{t-1}| (Eq. 1) from
// N-bit selection masks.  The directory update (App. A.1-A.2: hits and misses judged against
// the state before the step, then serve-and-admit with LRU/FIFO/LFU victims) is integer
// work done by one warp per layer, with one cache slot per lane during victim search.
#include "remoe_internal.cuh"

#include <math_constants.h>

namespace remoe {

namespace {

constexpr unsigned kFull = 0xffffffffu;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(kFull, v, o);
  return v;
}

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(kFull, v, o));
  return v;
}

// Dot product of one weight row (H <= 2048 elements, 16-byte aligned) with h (staged in shared memory),
// by one warp.  All of a lane's 16-byte pieces of the row (at most 8) are requested before the first is
// used, so a row costs one memory round trip instead of one per piece.
constexpr int kRowPieces = 8;
__device__ __forceinline__ float row_dot(const char* row, const float* __restrict__ h, int H,
                                         int wbytes, int lane) {
  float acc = 0.f;
  const uint4* r4 = reinterpret_cast<const uint4*>(row);
  const float4* h4 = reinterpret_cast<const float4*>(h);
  const int n = H * wbytes / 16;                     // 16-byte pieces in the row: <= 256
  uint4 w[kRowPieces];
#pragma unroll
  for (int i = 0; i < kRowPieces; ++i) {
    const int c = lane + 32 * i;
    w[i] = c < n ? __ldg(r4 + c) : make_uint4(0u, 0u, 0u, 0u);
  }
  if (wbytes == 4) {
#pragma unroll
    for (int i = 0; i < kRowPieces; ++i) {
      const int c = lane + 32 * i;
      if (c < n) {
        const float4 x = h4[c];
        acc = fmaf(__uint_as_float(w[i].x), x.x, acc);
        acc = fmaf(__uint_as_float(w[i].y), x.y, acc);
        acc = fmaf(__uint_as_float(w[i].z), x.z, acc);
        acc = fmaf(__uint_as_float(w[i].w), x.w, acc);
      }
    }
  } else {
#pragma unroll
    for (int i = 0; i < kRowPieces; ++i) {
      const int c = lane + 32 * i;
      if (c < n) {
        const float4 x0 = h4[2 * c], x1 = h4[2 * c + 1];
        acc = fmaf(__uint_as_float(w[i].x << 16), x0.x, acc);
        acc = fmaf(__uint_as_float(w[i].x & 0xffff0000u), x0.y, acc);
        acc = fmaf(__uint_as_float(w[i].y << 16), x0.z, acc);
        acc = fmaf(__uint_as_float(w[i].y & 0xffff0000u), x0.w, acc);
        acc = fmaf(__uint_as_float(w[i].z << 16), x1.x, acc);
        acc = fmaf(__uint_as_float(w[i].z & 0xffff0000u), x1.y, acc);
        acc = fmaf(__uint_as_float(w[i].w << 16), x1.z, acc);
        acc = fmaf(__uint_as_float(w[i].w & 0xffff0000u), x1.w, acc);
      }
    }
  }
  return warp_sum(acc);
}

struct DirSmem {
  unsigned long long stamp[kMaxSlots];
  int eos[kMaxSlots];
  unsigned freq[kMaxSlots];
  int soe[kMaxRouted];
  int uniq[kMaxRequests];
  unsigned char hitf[kMaxRequests];
  unsigned seen[kMaskWords];
  int uidx[kMaxRouted];                 // position of an expert in the unique list
  int gcnt[kMaxRequests];               // tokens collected so far per unique request
  unsigned char sgen[kMaxSlots];        // this step's occupants a slot has had so far
};

// Cache resolution for one layer by one warp.  `flat` holds the step's B*K requested ids in
// (sequence, rank) order (App. E.2.3: R); U = Unique(R) keeps first occurrences.
// The layer's directory as it stands before the step, into shared memory (one warp).
__device__ __forceinline__ void load_directory(const DevStack& d, int l, DirSmem& sm, int lane) {
  const int C = d.C, N = d.N;
  for (int s = lane; s < C; s += 32) {
    sm.sgen[s] = 0;
    sm.eos[s] = d.expert_of_slot[l * C + s];
    sm.stamp[s] = d.stamp[l * C + s];
    sm.freq[s] = d.freq[l * C + s];
  }
  for (int e = lane; e < N; e += 32) sm.soe[e] = d.slot_of_expert[l * N + e];
  if (lane < kMaskWords) sm.seen[lane] = 0u;
}

__device__ void resolve_layer(const DevStack& d, int l, const int* flat, int n_flat, DirSmem& sm,
                              int lane, int* contrib, bool directory_loaded = false) {
  const int C = d.C, N = d.N, BK = d.B * d.K;
  if (!directory_loaded) load_directory(d, l, sm, lane);
  __syncwarp();

  const unsigned lt = (1u << lane) - 1u;
  int n_u = 0, tok_h = 0;
  for (int base = 0; base < n_flat; base += 32) {
    const int i = base + lane;
    const bool valid = i < n_flat;
    int e = valid ? flat[i] : -1 - lane;
    if (valid && (e < 0 || e >= N)) { atomicCAS(d.err, kErrNone, kErrBadIndex); e = 0; }
    const bool resident = valid && sm.soe[e] >= 0;
    if (valid) atomicAdd(d.load + (size_t)l * N + e, 1ull);     // expert load (integer: order-free)
    tok_h += __popc(__ballot_sync(kFull, resident));
    const unsigned same = __match_any_sync(kFull, e);
    const bool first_here = valid && (__ffs(same) - 1 == lane);
    const bool seen_before = valid && ((sm.seen[e >> 5] >> (e & 31)) & 1u);
    const bool is_new = first_here && !seen_before;
    const unsigned newmask = __ballot_sync(kFull, is_new);
    if (is_new) {
      sm.uniq[n_u + __popc(newmask & lt)] = e;
      atomicOr(&sm.seen[e >> 5], 1u << (e & 31));
    }
    n_u += __popc(newmask);
    __syncwarp();
  }

  int* t_req = trace_requests(d.trace, d.L, BK) + l * BK;
  int* t_hit = trace_hit(d.trace, d.L, BK) + l * BK;
  int* t_slot = trace_slot(d.trace, d.L, BK) + l * BK;
  int* t_ev = trace_evicted(d.trace, d.L, BK) + l * BK;
  int* t_depth = trace_depth(d.trace, d.L, BK) + l * BK;

  if (d.B > 1) {
    // Token groups: for every distinct request, the sequences that selected it (ascending)
    // and the rank at which they did.
    for (int i = lane; i < n_u; i += 32) { sm.uidx[sm.uniq[i]] = i; sm.gcnt[i] = 0; }
    __syncwarp();
    for (int base = 0; base < n_flat; base += 32) {
      const int f = base + lane;
      const bool valid = f < n_flat;
      const int ui = valid ? sm.uidx[flat[f]] : -1 - lane;
      const unsigned same = __match_any_sync(kFull, ui);
      if (valid) {
        const int pos = sm.gcnt[ui] + __popc(same & lt);
        const size_t g = ((size_t)l * BK + ui) * d.B + pos;
        d.grp_tok[g] = f / d.K;
        d.grp_k[g] = f % d.K;
      }
      __syncwarp();
      if (valid && (__ffs(same) - 1 == lane)) sm.gcnt[ui] += __popc(same);
      __syncwarp();
    }
    for (int i = lane; i < BK; i += 32) d.grp_count[l * BK + i] = i < n_u ? sm.gcnt[i] : 0;
  }

  // Classification against the pre-step state, then phase 1: touch hits in request order.
  unsigned long long clock = d.clock[l];
  int uniq_h = 0;
  for (int base = 0; base < BK; base += 32) {
    const int i = base + lane;
    const bool valid = i < n_u;
    const int e = valid ? sm.uniq[i] : -1;
    const int s = valid ? sm.soe[e] : -1;
    const bool hit = s >= 0;
    const unsigned hm = __ballot_sync(kFull, hit);
    if (hit) {
      if (d.policy != REMOE_POLICY_FIFO) sm.stamp[s] = clock + 1 + __popc(hm & lt);
      sm.freq[s] += 1u;
      sm.sgen[s] = 1;
    }
    clock += __popc(hm);
    uniq_h += __popc(hm);
    if (i < BK) {
      t_req[i] = e;
      t_hit[i] = valid ? (hit ? 1 : 0) : 0;
      t_slot[i] = s;
      t_ev[i] = -1;
      t_depth[i] = 0;
      sm.hitf[i] = hit ? 1 : 0;
    }
    __syncwarp();
  }

  // Phase 2: admit misses in request order.  Victim: lowest empty slot; else the oldest
  // (LFU: least used, then oldest) occupant that is not part of this step's request; only if
  // every slot holds one of this step's experts, the oldest of all.
  for (int i = 0; i < n_u; ++i) {
    if (sm.hitf[i]) continue;
    const int e = sm.uniq[i];
    unsigned long long best = ~0ull;
    int best_s = -1;
    for (int s = lane; s < C; s += 32) {
      const int occ = sm.eos[s];
      unsigned long long key;
      if (occ < 0) {
        key = (unsigned long long)s;
      } else {
        const unsigned long long cls = ((sm.seen[occ >> 5] >> (occ & 31)) & 1u) ? 2ull : 1ull;
        const unsigned long long f =
            d.policy == REMOE_POLICY_LFU ? (unsigned long long)min(sm.freq[s], 0x3fffffu) : 0ull;
        key = (cls << 62) | (f << 40) | (sm.stamp[s] & ((1ull << 40) - 1ull));
      }
      if (key < best) { best = key; best_s = s; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const unsigned long long ok = __shfl_xor_sync(kFull, best, o);
      const int os = __shfl_xor_sync(kFull, best_s, o);
      if (os >= 0 && (best_s < 0 || ok < best || (ok == best && os < best_s))) { best = ok; best_s = os; }
    }
    if (lane == 0) {
      const int ev = sm.eos[best_s];
      if (ev >= 0) sm.soe[ev] = -1;
      sm.eos[best_s] = e;
      sm.soe[e] = best_s;
      clock += 1;
      sm.stamp[best_s] = clock;
      sm.freq[best_s] = 1u;
      t_slot[i] = best_s;
      t_ev[i] = ev;
      t_depth[i] = sm.sgen[best_s];
      sm.sgen[best_s] += 1;
    }
    __syncwarp();
  }

  for (int s = lane; s < C; s += 32) {
    d.expert_of_slot[l * C + s] = sm.eos[s];
    d.stamp[l * C + s] = sm.stamp[s];
    d.freq[l * C + s] = sm.freq[s];
  }
  for (int e = lane; e < N; e += 32) d.slot_of_expert[l * N + e] = sm.soe[e];
  if (lane == 0) {
    d.clock[l] = clock;
    unsigned long long* c = d.counters + (size_t)l * kCounters;
    c[0] += (unsigned long long)tok_h;
    c[1] += (unsigned long long)(n_flat - tok_h);
    c[2] += (unsigned long long)uniq_h;
    c[3] += (unsigned long long)(n_u - uniq_h);
    trace_n_unique(d.trace)[l] = n_u;
    trace_tok_hits(d.trace, d.L, BK)[l] = tok_h;
    contrib[(d.L + l) * 2 + 0] = 1;      // no miss-phase contribution yet for this layer
    contrib[(d.L + l) * 2 + 1] = 0;
  }
  if (d.host_mirror) {
    // this layer's part of the trace, and the error word if set, straight to mapped host memory
    __syncwarp();
    int* ht = d.host_mirror + 1;
    for (int i = lane; i < BK; i += 32) {
      trace_requests(ht, d.L, BK)[l * BK + i] = t_req[i];
      trace_hit(ht, d.L, BK)[l * BK + i] = t_hit[i];
      trace_slot(ht, d.L, BK)[l * BK + i] = t_slot[i];
      trace_evicted(ht, d.L, BK)[l * BK + i] = t_ev[i];
      trace_depth(ht, d.L, BK)[l * BK + i] = t_depth[i];
    }
    if (lane == 0) {
      trace_n_unique(ht)[l] = n_u;
      trace_tok_hits(ht, d.L, BK)[l] = tok_h;
      const int e = *(volatile int*)d.err;
      if (e != kErrNone) d.host_mirror[0] = e;
    }
    __threadfence_system();
  }
}

// Shared memory of one routing CTA.
struct RouteSmem {
  float z[kMaxRouted];
  int ids[32];
  float g[32];
  __align__(16) float h[kMaxHidden];
  DirSmem dir;
};

// Routing of one (layer, sequence) by one CTA whose input vector is already in sm.h: router logits (one warp
// per expert row), shared-expert gate, then, by warp 0, softmax, top-K, gate weights, reuse statistics and,
// at batch 1, the cache directory update.  Every thread of the CTA must call it.
__device__ void route_block(const DevStack& d, RouteSmem& sm, int lb, int* __restrict__ ids,
                            float* __restrict__ gates, int* contrib) {
  float* z = sm.z;
  int* s_ids = sm.ids;
  float* s_g = sm.g;
  const float* h = sm.h;
  const int l = lb / d.B;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const size_t row_bytes = (size_t)d.H * d.rbytes;

  const int n_warps = blockDim.x >> 5;
  // at batch 1 the directory update follows in this CTA: one warp fetches the directory image while the
  // others are waiting for their router rows, so that round trip is off the resolve warp's chain
  const bool preload = d.B == 1 && n_warps >= 3;
  if (preload && warp == n_warps - 2) load_directory(d, l, sm.dir, lane);
  for (int e = warp; e < d.N; e += n_warps) {
    const float acc = row_dot(d.router + ((size_t)l * d.N + e) * row_bytes, h, d.H, d.rbytes, lane);
    if (lane == 0) z[e] = acc;
  }
  if (warp == n_warps - 1) {
    float sc = 1.f;
    if (d.shared_gate) {
      const float dot = row_dot(d.shared_gate_w + (size_t)l * row_bytes, h, d.H, d.rbytes, lane);
      sc = 1.f / (1.f + expf(-dot));
    }
    if (lane == 0) d.shared_scale[lb] = sc;
  }
  __syncthreads();
  if (warp != 0) return;
  // Softmax over all N logits and top-K on the (optionally residency-biased) logits.
  float v[kMaskWords], sc[kMaskWords];
  float m = -CUDART_INF_F;
#pragma unroll
  for (int j = 0; j < kMaskWords; ++j) {
    const int e = lane + 32 * j;
    v[j] = e < d.N ? z[e] : -CUDART_INF_F;
    sc[j] = v[j];
    if (d.beta != 0.f && e < d.N && (preload ? sm.dir.soe[e] : d.slot_of_expert[l * d.N + e]) >= 0) sc[j] += d.beta;
    m = fmaxf(m, v[j]);
  }
  m = warp_max(m);
  float sum = 0.f;
#pragma unroll
  for (int j = 0; j < kMaskWords; ++j)
    if (lane + 32 * j < d.N) sum += expf(v[j] - m);
  sum = warp_sum(sum);

  unsigned taken = 0u;
  for (int k = 0; k < d.K; ++k) {
    float best = -CUDART_INF_F;
    int idx = INT_MAX;
#pragma unroll
    for (int j = 0; j < kMaskWords; ++j) {
      const int e = lane + 32 * j;
      if (e < d.N && !((taken >> j) & 1u) && (idx == INT_MAX || sc[j] > best)) { best = sc[j]; idx = e; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ob = __shfl_xor_sync(kFull, best, o);
      const int oi = __shfl_xor_sync(kFull, idx, o);
      if (oi != INT_MAX && (idx == INT_MAX || ob > best || (ob == best && oi < idx))) { best = ob; idx = oi; }
    }
    if ((idx & 31) == lane) taken |= 1u << (idx >> 5);
    if (lane == 0) {
      s_ids[k] = idx;
      s_g[k] = expf(z[idx] - m) / sum;
    }
  }
  __syncwarp();
  if (lane == 0 && d.renorm) {
    float t = 0.f;
    for (int k = 0; k < d.K; ++k) t += s_g[k];
    for (int k = 0; k < d.K; ++k) s_g[k] /= t;
  }
  __syncwarp();
  if (lane < d.K) {
    ids[(size_t)lb * d.K + lane] = s_ids[lane];
    gates[(size_t)lb * d.K + lane] = s_g[lane];
  }

  // Reuse: |E_t n E_{t-1}| from selection bit masks (Eq. 1) and the reuse mass
  // m_t = (1/K) sum_{k in E_{t-1}} P_t^(k) (Eq. 2); both counted from the second step on.
  // The previous step's mask words are read in one round trip (lane j holds word j) and handed round by
  // shuffle; the new words go back the same way.
  int ov = 0;
  float mass = 0.f;
  unsigned* pm = d.prev_mask + (size_t)lb * kMaskWords;
  const unsigned prev_mine = (d.has_prev && lane < kMaskWords) ? pm[lane] : 0u;
  unsigned word_mine = 0u;
#pragma unroll
  for (int j = 0; j < kMaskWords; ++j) {
    const unsigned word = __ballot_sync(kFull, (taken >> j) & 1u);
    const unsigned prev = __shfl_sync(kFull, prev_mine, j);
    if ((prev >> lane) & 1u) mass += expf(v[j] - m) / sum;
    ov += __popc(word & prev);
    if (lane == j) word_mine = word;
  }
  if (lane < kMaskWords) pm[lane] = word_mine;
  mass = warp_sum(mass) / (float)d.K;
  if (lane == 0) {
    d.last_overlap[lb] = d.has_prev ? ov : -1;
    d.last_mass[lb] = d.has_prev ? mass : -1.f;
    if (d.has_prev) {
      d.mass_sum[lb] += (double)mass;
      atomicAdd(d.counters + (size_t)l * kCounters + 4, (unsigned long long)ov);
      atomicAdd(d.counters + (size_t)l * kCounters + 5, 1ull);
    }
  }
  if (d.B == 1) resolve_layer(d, l, s_ids, d.K, sm.dir, lane, contrib, preload);
}


__global__ void __launch_bounds__(1024) route_kernel(DevStack d, const float* __restrict__ hidden_in,
                                                    int* __restrict__ ids, float* __restrict__ gates,
                                                    int* contrib, int layer0) {
  __shared__ RouteSmem sm;
  const int lb = layer0 * d.B + blockIdx.x;
  for (int c = threadIdx.x; c < d.H / 4; c += blockDim.x)
    reinterpret_cast<float4*>(sm.h)[c] = __ldg(reinterpret_cast<const float4*>(hidden_in + (size_t)lb * d.H) + c);
  __syncthreads();
  route_block(d, sm, lb, ids, gates, contrib);
}

// Link between two layers of the chained batch-1 step, one launch instead of four: the fixed-order sum of
// layer (layer - 1)'s partial rows (the work of combine_kernel), the residual add h_layer = h_{layer-1} + out,
// the pre-norm x = h / sqrt(mean(h^2) + 1e-6) and the routing of `layer` on x.
//   grid = kLinkCtas CTAs of 1024 threads.  CTA c sums 1/kLinkCtas of the columns: 16 row groups of 64 threads,
//   a thread adding the float4 pieces of its group's rows in order, the groups then added in order (fixed
//   order, no float atomics).  The CTA that finishes last (a ticket counter; nobody waits for anybody) reads the
//   complete h back, normalises it and routes.  With do_combine == 0 (first layer) one CTA normalises and
//   routes h as it stands; with do_route == 0 (after the last layer) the sum and the residual add are all.
constexpr int kLinkCtas = 8;
struct LinkArgs {
  const float* partial;       // [2][L][grid_cap][H]
  const int* contrib_in;      // [2][L][2]
  int grid_cap;
  int layer;                  // layer to route; the partials summed are those of layer - 1
  float* chain_in;            // [L + 1][H] residual stream
  float* chain_out;           // [L][H] per-layer MoE outputs
  float* chain_x;             // [L][H] normalised layer inputs
  unsigned* ticket;
  int do_combine, do_route;
};

__global__ void __launch_bounds__(1024) chain_link_kernel(DevStack d, LinkArgs a, int* __restrict__ ids,
                                                         float* __restrict__ gates, int* contrib) {
  __shared__ RouteSmem sm;
  __shared__ float4 red[16][64];
  __shared__ int s_last;
  __shared__ float warp_ss[32];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int H = d.H, l = a.layer;

  if (a.do_combine) {
    const int lp = l - 1;
    const int cols = H / kLinkCtas;                       // columns of this CTA; H / 8 <= 256, a multiple of 4
    const int c4 = tid & 63, rg = tid >> 6;
    const int col = blockIdx.x * cols + c4 * 4;
    const bool active = c4 * 4 < cols;
    // rows: resident-phase partials lo0..hi0, then miss-phase partials lo1..hi1
    const int lo0 = a.contrib_in[(0 * d.L + lp) * 2], hi0 = a.contrib_in[(0 * d.L + lp) * 2 + 1];
    const int lo1 = a.contrib_in[(1 * d.L + lp) * 2], hi1 = a.contrib_in[(1 * d.L + lp) * 2 + 1];
    const int n0 = hi0 >= lo0 ? hi0 - lo0 + 1 : 0, n1 = hi1 >= lo1 ? hi1 - lo1 + 1 : 0;
    const int n = n0 + n1, per = (n + 15) / 16;
    const int ra = min(n, rg * per), rb = min(n, ra + per);
    float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
    if (active) {
      const float* p0 = a.partial + ((size_t)(0 * d.L + lp) * a.grid_cap) * H + col;
      const float* p1 = a.partial + ((size_t)(1 * d.L + lp) * a.grid_cap) * H + col;
#pragma unroll 8
      for (int r = ra; r < rb; ++r) {
        const float* src = r < n0 ? p0 + (size_t)(lo0 + r) * H : p1 + (size_t)(lo1 + r - n0) * H;
        const float4 v = __ldcg(reinterpret_cast<const float4*>(src));
        t.x += v.x; t.y += v.y; t.z += v.z; t.w += v.w;
      }
    }
    red[rg][c4] = t;
    __syncthreads();
    if (rg == 0 && active) {
      float4 o = red[0][c4];
#pragma unroll
      for (int g2 = 1; g2 < 16; ++g2) { o.x += red[g2][c4].x; o.y += red[g2][c4].y; o.z += red[g2][c4].z; o.w += red[g2][c4].w; }
      *reinterpret_cast<float4*>(a.chain_out + (size_t)lp * H + col) = o;
      const float4 hp = *reinterpret_cast<const float4*>(a.chain_in + (size_t)lp * H + col);
      *reinterpret_cast<float4*>(a.chain_in + (size_t)l * H + col) =
          make_float4(hp.x + o.x, hp.y + o.y, hp.z + o.z, hp.w + o.w);
    }
    // the CTA that takes the last ticket sees every other CTA's columns (fence, then ticket)
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const unsigned t0 = atomicAdd(a.ticket, 1u);
      s_last = t0 == gridDim.x - 1 ? 1 : 0;
      if (s_last) *a.ticket = 0u;                          // ready for the next launch
    }
    __syncthreads();
    if (!s_last || !a.do_route) return;
    __threadfence();
  }

  // pre-norm of h_l (fixed summation order), x_l to shared memory for the router and to global memory for
  // the expert kernels
  const float* hl = a.chain_in + (size_t)l * H;
  float ss = 0.f;
  for (int c = tid; c < H; c += 1024) {
    const float v = __ldcg(hl + c);
    sm.h[c] = v;
    ss = fmaf(v, v, ss);
  }
  ss = warp_sum(ss);
  if (lane == 0) warp_ss[warp] = ss;
  __syncthreads();
  float tot = 0.f;
  for (int w = 0; w < 32; ++w) tot += warp_ss[w];
  const float sc = rsqrtf(tot / (float)H + 1e-6f);
  for (int c = tid; c < H; c += 1024) {
    const float x = sm.h[c] * sc;
    sm.h[c] = x;
    a.chain_x[(size_t)l * H + c] = x;
  }
  __syncthreads();
  route_block(d, sm, l, ids, gates, contrib);
}

__global__ void __launch_bounds__(32) resolve_kernel(DevStack d, const int* __restrict__ ids, int* contrib,
                                                     int layer0) {
  __shared__ DirSmem dir;
  __shared__ int flat[kMaxRequests];
  const int l = layer0 + blockIdx.x, lane = threadIdx.x;
  const int BK = d.B * d.K;
  for (int i = lane; i < BK; i += 32) flat[i] = ids[(size_t)l * BK + i];
  __syncwarp();
  resolve_layer(d, l, flat, BK, dir, lane, contrib);
}

}  // namespace

cudaError_t launch_route(const DevStack& d, const float* hidden_in, int* ids, float* gates,
                         int* contrib, int layer0, int n_layers, cudaStream_t st) {
  // few CTAs at batch 1: give each as many warps as it can hold so the router rows load in parallel
  route_kernel<<<n_layers * d.B, d.B == 1 ? 1024 : 256, 0, st>>>(d, hidden_in, ids, gates, contrib, layer0);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (d.B > 1) {
    resolve_kernel<<<n_layers, 32, 0, st>>>(d, ids, contrib, layer0);
    e = cudaGetLastError();
  }
  return e;
}

// Chained batch-1 step: sum of layer (layer - 1)'s partials + residual add (do_combine), then pre-norm and
// routing of `layer` (do_route), in one launch.  `ticket` is one zero-initialised word owned by the stack.
cudaError_t launch_chain_link(const DevStack& d, const FfnArgs& f, int layer, float* chain_in, float* chain_out,
                              float* chain_x, unsigned* ticket, int do_combine, int do_route, int* ids, float* gates,
                              cudaStream_t st) {
  LinkArgs a{};
  a.partial = f.partial;
  a.contrib_in = f.contrib;
  a.grid_cap = f.grid_cap;
  a.layer = layer;
  a.chain_in = chain_in;
  a.chain_out = chain_out;
  a.chain_x = chain_x;
  a.ticket = ticket;
  a.do_combine = do_combine;
  a.do_route = do_route;
  chain_link_kernel<<<do_combine ? kLinkCtas : 1, 1024, 0, st>>>(d, a, ids, gates, f.contrib);
  return cudaGetLastError();
}

}  // namespace remoe

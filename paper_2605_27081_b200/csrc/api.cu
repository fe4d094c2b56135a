// Host side of libremoe: stack state, the per-step scheduler with its miss-fetch engine,
// statistics, and the extern "C" boundary declared in remoe.h.
//
// Per decode step (batch 1):
//   compute stream : route+resolve kernel (its resolve warps also write the step trace to a mirror in
//                    mapped page-locked host memory)
//                    -> resident-phase streaming kernel (hits + shared experts, all layers)
//   host           : waits only for the route kernel, then walks the mirrored trace: for each layer, one
//                    cudaMemcpyAsync per missing expert from its pinned host block into the
//                    victim slot on the copy stream, an event after the layer's last copy
//   compute stream : per layer with misses: wait for that event, miss-phase streaming kernel
//                    over the freshly filled slots; finally the combine kernel.
// Copies of later layers overlap the compute of earlier ones; nothing is ever inserted into a
// slot except the misses of an already routed step (no speculative prefetch, which would
// break the fetch bound of Prop. 3.1).
#include "remoe_internal.cuh"
#include "order_ledger.h"

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <memory>
#include <new>
#include <string>
#include <vector>

using namespace remoe;

struct EvPair {
  cudaEvent_t a, b;
  uint64_t bytes;
  int phase;
};

struct remoe_stack {
  remoe_shape shape{};
  int C = 0, device = 0, grid = 0, BK = 0;
  cudaStream_t stream = nullptr, copy_stream = nullptr;
  DevStack d{};
  std::vector<void*> dev_allocs;
  std::vector<void*> host_allocs;
  std::vector<const void*> host_ptrs;      // [L*N] borrowed pinned expert blocks
  std::vector<char> router_loaded, shared_loaded;
  int* dev_block = nullptr;                // [err | trace]
  int* host_block = nullptr;               // pinned mirror of dev_block
  size_t block_ints = 0;
  float* partial = nullptr;
  int* contrib = nullptr;
  float* chain_in = nullptr;               // [L + 1][H] residual stream h_l of the chained mode
  float* chain_x = nullptr;                // [L][H] normalised layer inputs x_l = rmsnorm(h_l)
  float* chain_out = nullptr;              // [L][H] per-layer MoE outputs of the chained mode
  unsigned* link_ticket = nullptr;         // ticket word of the chained step's link kernel
  cudaEvent_t ev_trace = nullptr;
  std::vector<cudaEvent_t> ev_layer;
  // second set of per-step buffers and the streams/events of the multi-step entry point, which routes
  // step t+1 while step t is still fetching and computing (created on first use)
  bool pipe_ready = false;
  cudaStream_t route_stream = nullptr;
  int* dev_block2 = nullptr;
  int* host_block2 = nullptr;
  int* contrib2 = nullptr;
  float* shared_scale2 = nullptr;
  cudaEvent_t ev_entry = nullptr, ev_route2[2] = {nullptr, nullptr}, ev_free2[2] = {nullptr, nullptr},
              ev_res2[2] = {nullptr, nullptr};
  std::vector<cudaEvent_t> ev_copy2, ev_miss2;     // [2][L]
  // batched path (B > 1)
  float* part = nullptr;
  int* flags = nullptr;
  int* plan = nullptr;
  int max_items = 0;
  int step_serial = 0;                    // never reset: stamps partial rows
  cudaEvent_t ev_resident = nullptr;
  bool use_tc = false;                     // batched experts on tcgen05 / TMEM, slots in operand-tile order
  bool widen_fp8 = false;                  // batched stack over an FP8 / 4-bit host store: blocks are widened to bf16 on arrival
  int host_wbytes = 0;                     // element tag of the host store (see weight_row_bytes)
  size_t fetch_bytes = 0, fetch_shared_bytes = 0;   // bytes of one routed / shared expert block in HOST memory
  char* stage_pool = nullptr;              // [2][C] channel-major landing area of fetched blocks (use_tc)
  size_t stage_bytes = 0;
  cudaEvent_t ev_stage[2] = {nullptr, nullptr};   // retile of the group that last used a half is enqueued
  bool stage_used[2] = {false, false};
  uint64_t stage_group = 0;                // running (depth, layer) group number: picks the half
  alignas(64) unsigned char tc_maps[1024];
  std::vector<cudaEvent_t> ev_pool;        // copy-done / compute-done events of the waves
  uint64_t steps = 0, steps_since_reset = 0;
  std::vector<uint64_t> h2d_bytes;         // per layer
  std::vector<uint32_t> hist_umiss, hist_tok_hits;   // per step since the last reset, summed over layers
  // staging for the host-buffer entry point
  float *st_in_d = nullptr, *st_out_d = nullptr, *st_g_d = nullptr;
  int* st_ids_d = nullptr;
  float *st_in_h = nullptr, *st_out_h = nullptr, *st_g_h = nullptr;
  int* st_ids_h = nullptr;
  // profiling
  bool profiling = false;
  std::vector<EvPair> ev_used, ev_free;
  double prof_ms[2] = {0.0, 0.0};
  uint64_t prof_launches[2] = {0, 0}, prof_bytes[2] = {0, 0};
  uint64_t kernel_launches = 0;          // every kernel this stack has launched
  std::string cuda_err;
  // failure-detection test aid (REMOE_FAULT_INJECT=lost_copy at creation): the first resident-phase launch
  // of the batch-1 step runs with a short wait limit and one weight row whose copy is never issued
  bool inject_lost_copy = false;
  // REMOE_CHECK_ORDER=1 at creation: every decode call also replays what it enqueues (operations, event
  // records and waits, host waits) into a ledger that checks that each write of a cache slot is ordered
  // behind the readers of the slot's previous contents and each read behind the write that filled it
  std::unique_ptr<OrderLedger> ledger;
  uint64_t ledger_reported = 0;
  int policy = REMOE_POLICY_LRU;
  float beta = 0.f;
};

namespace {

int fail_cuda(remoe_stack* s, cudaError_t e, const char* what) {
  if (s) {
    s->cuda_err = std::string(what) + ": " + cudaGetErrorString(e);
  }
  return REMOE_E_CUDA;
}

#define CK(call)                                                    \
  do {                                                              \
    cudaError_t e_ = (call);                                        \
    if (e_ != cudaSuccess) return fail_cuda(s, e_, #call);          \
  } while (0)

// Makes the stack's device current for the duration of a call and puts the caller's back afterwards.
struct DeviceGuard {
  int prev = -1;
  bool switched = false;
  cudaError_t err = cudaSuccess;
  explicit DeviceGuard(int dev) {
    err = cudaGetDevice(&prev);
    if (err == cudaSuccess && prev != dev) {
      err = cudaSetDevice(dev);
      switched = err == cudaSuccess;
    }
  }
  ~DeviceGuard() {
    if (switched) cudaSetDevice(prev);
  }
  DeviceGuard(const DeviceGuard&) = delete;
  DeviceGuard& operator=(const DeviceGuard&) = delete;
};
#define ON_STACK_DEVICE(s)                                                       \
  DeviceGuard device_guard_((s)->device);                                        \
  if (device_guard_.err != cudaSuccess) return fail_cuda((s), device_guard_.err, "cudaSetDevice")

// ---- ordering ledger hooks (no-ops unless the stack was created with REMOE_CHECK_ORDER=1)
enum { kStCompute = 0, kStCopy = 1, kStRoute = 2 };
using LOp = OrderLedger::Op;
inline LOp l_op(remoe_stack* s, int st) { return s->ledger ? s->ledger->op(st) : LOp{}; }
inline void l_record(remoe_stack* s, const void* ev, int st) { if (s->ledger) s->ledger->record(ev, st); }
inline void l_wait(remoe_stack* s, int st, const void* ev) { if (s->ledger) s->ledger->wait(st, ev); }
inline void l_host_wait(remoe_stack* s, const void* ev) { if (s->ledger) s->ledger->host_wait(ev); }
inline void l_host_sync(remoe_stack* s, int st) { if (s->ledger) s->ledger->host_sync(st); }
inline void l_read(remoe_stack* s, const LOp& o, uint64_t cell, const char* what) { if (s->ledger) s->ledger->read(o, cell, what); }
inline void l_write(remoe_stack* s, const LOp& o, uint64_t cell, const char* what) { if (s->ledger) s->ledger->write(o, cell, what); }
inline uint64_t slot_cell(const remoe_stack* s, int l, int slot) { return (uint64_t)l * s->d.C + slot; }
inline uint64_t stage_cell(const remoe_stack* s, int half, int i) { return (1ull << 40) + (uint64_t)half * s->d.C + i; }
// New violations since the last call end the call with REMOE_E_ORDER.
int l_verdict(remoe_stack* s) {
  if (!s->ledger || s->ledger->violations() == s->ledger_reported) return REMOE_OK;
  s->ledger_reported = s->ledger->violations();
  s->cuda_err = "schedule order: " + s->ledger->first_violation();
  return REMOE_E_ORDER;
}

template <typename T>
int dev_alloc(remoe_stack* s, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t e = cudaMalloc(&q, count * sizeof(T) > 0 ? count * sizeof(T) : 16);
  if (e != cudaSuccess) {
    fail_cuda(s, e, "cudaMalloc");
    return e == cudaErrorMemoryAllocation ? REMOE_E_NOMEM : REMOE_E_CUDA;
  }
  s->dev_allocs.push_back(q);
  *p = static_cast<T*>(q);
  return REMOE_OK;
}

template <typename T>
int host_alloc(remoe_stack* s, T** p, size_t count) {
  void* q = nullptr;
  cudaError_t e = cudaMallocHost(&q, count * sizeof(T) > 0 ? count * sizeof(T) : 16);
  if (e != cudaSuccess) {
    fail_cuda(s, e, "cudaMallocHost");
    return REMOE_E_NOMEM;
  }
  s->host_allocs.push_back(q);
  *p = static_cast<T*>(q);
  return REMOE_OK;
}

int reset_state(remoe_stack* s) {
  const DevStack& d = s->d;
  const size_t L = d.L;
  CK(cudaMemsetAsync(d.expert_of_slot, 0xff, L * d.C * sizeof(int), s->stream));
  CK(cudaMemsetAsync(d.slot_of_expert, 0xff, L * d.N * sizeof(int), s->stream));
  CK(cudaMemsetAsync(d.stamp, 0, L * d.C * sizeof(unsigned long long), s->stream));
  CK(cudaMemsetAsync(d.freq, 0, L * d.C * sizeof(unsigned), s->stream));
  CK(cudaMemsetAsync(d.clock, 0, L * sizeof(unsigned long long), s->stream));
  CK(cudaMemsetAsync(d.prev_mask, 0, L * d.B * kMaskWords * sizeof(unsigned), s->stream));
  CK(cudaMemsetAsync(d.counters, 0, L * kCounters * sizeof(unsigned long long), s->stream));
  CK(cudaMemsetAsync(d.load, 0, L * d.N * sizeof(unsigned long long), s->stream));
  CK(cudaMemsetAsync(d.last_overlap, 0xff, L * d.B * sizeof(int), s->stream));
  CK(cudaMemsetAsync(d.last_mass, 0, L * d.B * sizeof(float), s->stream));
  CK(cudaMemsetAsync(d.mass_sum, 0, L * d.B * sizeof(double), s->stream));
  CK(cudaMemsetAsync(s->dev_block, 0, s->block_ints * sizeof(int), s->stream));
  CK(cudaStreamSynchronize(s->stream));
  l_host_sync(s, kStCompute);
  std::memset(s->host_block, 0, s->block_ints * sizeof(int));
  if (s->host_block2) std::memset(s->host_block2, 0, s->block_ints * sizeof(int));
  s->steps = 0;
  s->steps_since_reset = 0;
  std::fill(s->h2d_bytes.begin(), s->h2d_bytes.end(), 0);
  s->hist_umiss.clear();
  s->hist_tok_hits.clear();
  return REMOE_OK;
}

bool everything_loaded(const remoe_stack* s) {
  for (char c : s->router_loaded) if (!c) return false;
  for (char c : s->shared_loaded) if (!c) return false;
  for (const void* p : s->host_ptrs) if (!p) return false;
  return true;
}

int prof_begin(remoe_stack* s, cudaStream_t st, uint64_t bytes, int phase) {
  if (!s->profiling) return REMOE_OK;
  EvPair p;
  if (!s->ev_free.empty()) {
    p = s->ev_free.back();
    s->ev_free.pop_back();
  } else {
    CK(cudaEventCreate(&p.a));
    CK(cudaEventCreate(&p.b));
  }
  p.bytes = bytes;
  p.phase = phase;
  CK(cudaEventRecord(p.a, st));
  s->ev_used.push_back(p);
  return REMOE_OK;
}

int prof_end(remoe_stack* s, cudaStream_t st) {
  if (!s->profiling) return REMOE_OK;
  CK(cudaEventRecord(s->ev_used.back().b, st));
  return REMOE_OK;
}

int prof_collect(remoe_stack* s) {
  for (EvPair& p : s->ev_used) {
    float ms = 0.f;
    CK(cudaEventSynchronize(p.b));
    CK(cudaEventElapsedTime(&ms, p.a, p.b));
    s->prof_ms[p.phase] += ms;
    s->prof_launches[p.phase] += 1;
    s->prof_bytes[p.phase] += p.bytes;
    s->ev_free.push_back(p);
  }
  s->ev_used.clear();
  return REMOE_OK;
}

int check_device_flag(remoe_stack* s, const int* block = nullptr) {
  if (!block) block = s->host_block;
  if (block[0] == kErrNone) return REMOE_OK;
  static const char* names[] = {"none", "a consumer's bounded wait for a weight row ran out",
                                "the producer's bounded wait for a free stage ran out",
                                "an expert id or slot index was out of range",
                                "copies were still in flight when a kernel bailed out"};
  const int c = block[0];
  s->cuda_err = std::string("device flag ") + std::to_string(c) + ": " + (c >= 1 && c <= 4 ? names[c] : "unknown");
  return REMOE_E_DEVICE_FLAG;
}

// With the stack's stream drained: the device error word, which the expert and combine kernels of the
// last step may have set after the route kernel mirrored it to the host.
int fetch_device_flag(remoe_stack* s) {
  int e = kErrNone;
  CK(cudaMemcpy(&e, s->dev_block, sizeof(int), cudaMemcpyDeviceToHost));
  if (e == kErrNone) return REMOE_OK;
  s->host_block[0] = e;
  return check_device_flag(s);
}

// One decode step for B > 1.  The step's distinct requests may outnumber the slots, so a slot
// can be handed on within the step: its occupants are processed in "depth" order.  Depth-0
// experts are the cache hits (computed at once together with the shared experts) and the misses
// that displace experts nobody asked for in this step; a depth-d miss displaces a depth-(d-1)
// expert of this step and may only be copied once that one has been computed.  Copies are queued
// depth by depth, layer by layer, so the copy engine stays busy; each (depth, layer) group is
// computed as soon as its copies have landed.
cudaError_t launch_batched(remoe_stack* s, const BatchArgs& a) {
  return s->use_tc ? launch_ffn_batched_tc(a, s->grid, s->stream) : launch_ffn_batched(a, s->grid, s->stream);
}

// Validates the trace of layers [l0, l1) and runs their miss waves: copies queued depth by depth, layer
// by layer; each (depth, layer) group computed once its copies have landed.  The resident-phase launch
// covering these layers must already be enqueued with ev_resident recorded behind it.  Adds the
// algorithmic bytes of that launch to *resident_bytes.
int batched_waves(remoe_stack* s, BatchArgs& a, int l0, int l1, uint64_t* resident_bytes, const LOp& op_res) {
  DevStack& d = s->d;
  const int BK = s->BK;
  int* tr = s->host_block + 1;
  const int* t_nu = trace_n_unique(tr);
  const int* t_req = trace_requests(tr, d.L, BK);
  const int* t_hit = trace_hit(tr, d.L, BK);
  const int* t_slot = trace_slot(tr, d.L, BK);
  const int* t_depth = trace_depth(tr, d.L, BK);
  int max_depth = -1;
  for (int l = l0; l < l1; ++l) {
    if (t_nu[l] < 0 || t_nu[l] > BK) return REMOE_E_DEVICE_FLAG;
    for (int i = 0; i < t_nu[l]; ++i) {
      const int j = l * BK + i;
      if (t_hit[j]) {
        *resident_bytes += d.slot_bytes;
        if (t_slot[j] >= 0 && t_slot[j] < d.C) l_read(s, op_res, slot_cell(s, l, t_slot[j]), "resident-phase launch");
        continue;
      }
      if (t_req[j] < 0 || t_req[j] >= d.N || t_slot[j] < 0 || t_slot[j] >= d.C || t_depth[j] < 0)
        return REMOE_E_DEVICE_FLAG;
      if (t_depth[j] > max_depth) max_depth = t_depth[j];
    }
    *resident_bytes += (uint64_t)d.S * d.shared_bytes;   // algorithmic: once, although every token tile streams it
  }

  // events: [depth][layer] copy-done and compute-done
  const size_t need = (size_t)2 * (max_depth + 1) * d.L;
  while (s->ev_pool.size() < need) {
    cudaEvent_t e;
    CK(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    s->ev_pool.push_back(e);
  }
  auto ev_copy = [&](int dep, int l) { return s->ev_pool[((size_t)dep * d.L + l) * 2]; };
  auto ev_comp = [&](int dep, int l) { return s->ev_pool[((size_t)dep * d.L + l) * 2 + 1]; };
  std::vector<char> had(((size_t)max_depth + 2) * d.L, 0);

  // Channel-major slots (mma.sync kernel): a copy writes the slot itself, so it waits for every reader
  // of the slot's previous occupant.  Operand-tile-order slots (tcgen05 kernel): a copy lands in one
  // half of the staging pool and the retile kernel, on the compute stream behind those readers, writes
  // the slot; the copy engine then only ever waits for a staging half to be free.
  const bool staged = s->use_tc;
  if (max_depth >= 0 && !staged) {
    CK(cudaStreamWaitEvent(s->copy_stream, s->ev_trace, 0));
    l_wait(s, kStCopy, s->ev_trace);
  }
  std::vector<size_t> src_off;
  std::vector<char*> dst_ptr;
  std::vector<const void*> src_ptr;
  struct Fetch {
    const char* src;       // the expert's block in host memory
    char* slot;            // its cache slot
    int j;                 // its place in the trace
  };
  std::vector<Fetch> group;
  for (int dep = 0; dep <= max_depth; ++dep) {
    if (dep == 1 && !staged) {
      CK(cudaStreamWaitEvent(s->copy_stream, s->ev_resident, 0));   // displaced hits are done
      l_wait(s, kStCopy, s->ev_resident);
    }
    for (int l = l0; l < l1; ++l) {
      // one (depth, layer) group: its copies, then (enqueued at once, run when they have landed) its
      // retile and compute launches.  Streams keep the order depth-major, layer-minor.
      int misses = 0, half = 0;
      src_off.clear();
      dst_ptr.clear();
      group.clear();
      for (int i = 0; i < t_nu[l]; ++i) {
        const int j = l * BK + i;
        if (t_hit[j] || t_depth[j] != dep) continue;
        group.push_back({static_cast<const char*>(s->host_ptrs[(size_t)l * d.N + t_req[j]]),
                         d.slots + ((size_t)l * d.C + t_slot[j]) * d.slot_bytes, j});
      }
      if (staged && !group.empty()) {
        if ((int)group.size() > d.C) return REMOE_E_DEVICE_FLAG;   // more misses of one depth than slots: bad trace
        // the half's previous user is the group before last: its retile is already enqueued
        half = (int)(s->stage_group++ & 1);
        if (s->stage_used[half]) {
          CK(cudaStreamWaitEvent(s->copy_stream, s->ev_stage[half], 0));
          l_wait(s, kStCopy, s->ev_stage[half]);
        }
        // The landing places in the staging pool are ours to choose: the group's blocks are laid down in the
        // order of their host addresses, so blocks that are neighbours in host memory are neighbours in the pool
        // and go over the link as one copy (the copy engine loses a few microseconds per copy command).
        std::sort(group.begin(), group.end(), [](const Fetch& x, const Fetch& y) { return x.src < y.src; });
        for (size_t k = 0; k < group.size();) {
          size_t run = 1;
          while (k + run < group.size() && group[k + run].src == group[k].src + run * s->fetch_bytes) ++run;
          const size_t off = ((size_t)half * d.C + k) * s->fetch_bytes;
          CK(cudaMemcpyAsync(s->stage_pool + off, group[k].src, run * s->fetch_bytes, cudaMemcpyHostToDevice,
                             s->copy_stream));
          const LOp oc = l_op(s, kStCopy);
          for (size_t r = 0; r < run; ++r) {
            src_off.push_back(off + r * s->fetch_bytes);
            dst_ptr.push_back(group[k + r].slot);
            l_write(s, oc, stage_cell(s, half, (int)(k + r)), "miss fetch");
          }
          k += run;
        }
        misses = (int)group.size();
      } else {
        for (const Fetch& f : group) {
          if (!misses && dep >= 1 && had[(size_t)(dep - 1) * d.L + l]) {
            CK(cudaStreamWaitEvent(s->copy_stream, ev_comp(dep - 1, l), 0));        // displaced misses are done
            l_wait(s, kStCopy, ev_comp(dep - 1, l));
          }
          CK(cudaMemcpyAsync(f.slot, f.src, s->fetch_bytes, cudaMemcpyHostToDevice, s->copy_stream));
          l_write(s, l_op(s, kStCopy), slot_cell(s, l, t_slot[f.j]), "miss fetch");
          ++misses;
        }
      }
      if (!misses) continue;
      had[(size_t)dep * d.L + l] = 1;
      s->h2d_bytes[l] += (uint64_t)misses * s->fetch_bytes;
      CK(cudaEventRecord(ev_copy(dep, l), s->copy_stream));
      l_record(s, ev_copy(dep, l), kStCopy);

      CK(cudaStreamWaitEvent(s->stream, ev_copy(dep, l), 0));
      l_wait(s, kStCompute, ev_copy(dep, l));
      if (staged) {
        if (s->widen_fp8) {
          src_ptr.clear();
          for (size_t off : src_off) src_ptr.push_back(s->stage_pool + off);
          CK(launch_widen_retile_tc(d, s->host_wbytes, misses, src_ptr.data(), dst_ptr.data(), d.I, s->stream));
        } else {
          CK(launch_retile_tc(d, s->tc_maps, misses, src_off.data(), dst_ptr.data(), d.I, s->stream));
        }
        s->kernel_launches += (misses + 63) / 64;
        if (s->ledger) {
          const LOp ot = l_op(s, kStCompute);             // reads the staging half, rewrites the slots
          for (size_t k = 0; k < group.size(); ++k) {
            l_read(s, ot, stage_cell(s, half, (int)k), "retile");
            l_write(s, ot, slot_cell(s, l, t_slot[group[k].j]), "retile");
          }
        }
        CK(cudaEventRecord(s->ev_stage[half], s->stream));
        l_record(s, s->ev_stage[half], kStCompute);
        s->stage_used[half] = true;
      }
      a.phase = 1;
      a.layer = l;
      a.depth = dep;
      int rc = prof_begin(s, s->stream, (uint64_t)misses * d.slot_bytes, 1);
      if (rc != REMOE_OK) return rc;
      CK(launch_batched(s, a));
      s->kernel_launches += 2;
      if (s->ledger) {
        const LOp om = l_op(s, kStCompute);
        for (int i = 0; i < t_nu[l]; ++i) {
          const int j = l * BK + i;
          if (!t_hit[j] && t_depth[j] == dep) l_read(s, om, slot_cell(s, l, t_slot[j]), "miss-phase launch");
        }
      }
      rc = prof_end(s, s->stream);
      if (rc != REMOE_OK) return rc;
      CK(cudaEventRecord(ev_comp(dep, l), s->stream));
      l_record(s, ev_comp(dep, l), kStCompute);
    }
  }
  return REMOE_OK;
}

// #uMiss and token-level hits of layers [l0, l1) of the step whose trace is in the host block.
void trace_totals(const remoe_stack* s, int l0, int l1, uint32_t* umiss, uint32_t* tok_hits) {
  const int L = s->d.L, BK = s->BK;
  const int* th = trace_tok_hits(s->host_block + 1, L, BK);
  const int* nu = trace_n_unique(s->host_block + 1);
  const int* hh = trace_hit(s->host_block + 1, L, BK);
  for (int l = l0; l < l1; ++l) {
    *tok_hits += (uint32_t)th[l];
    for (int i = 0; i < nu[l] && i < BK; ++i) *umiss += hh[l * BK + i] ? 0u : 1u;
  }
}

int decode_step_batched(remoe_stack* s, const float* hin, float* hout, int32_t* ids, float* gates) {
  DevStack& d = s->d;
  d.has_prev = s->steps_since_reset > 0 ? 1 : 0;
  d.policy = s->policy;
  d.beta = s->beta;

  CK(launch_route(d, hin, ids, gates, s->contrib, 0, d.L, s->stream));
  s->kernel_launches += 2;
  l_op(s, kStCompute);
  CK(cudaEventRecord(s->ev_trace, s->stream));      // the route kernel has written the trace to the host mirror
  l_record(s, s->ev_trace, kStCompute);

  BatchArgs a{};
  a.d = d;
  a.hidden_in = hin;
  a.gates = gates;
  a.part = s->part;
  a.flags = s->flags;
  a.plan = s->plan;
  a.max_items = s->max_items;
  a.step_id = ++s->step_serial;
  a.phase = 0;
  a.layer = -1;
  a.depth = 0;
  int rc = prof_begin(s, s->stream, 0, 0);
  if (rc != REMOE_OK) return rc;
  CK(launch_batched(s, a));
  s->kernel_launches += 2;
  const LOp op_res = l_op(s, kStCompute);
  rc = prof_end(s, s->stream);
  if (rc != REMOE_OK) return rc;
  const size_t prof_slot = s->profiling ? s->ev_used.size() - 1 : 0;
  CK(cudaEventRecord(s->ev_resident, s->stream));
  l_record(s, s->ev_resident, kStCompute);

  CK(cudaEventSynchronize(s->ev_trace));
  l_host_wait(s, s->ev_trace);
  s->steps += 1;
  s->steps_since_reset += 1;
  if (check_device_flag(s) != REMOE_OK) return REMOE_E_DEVICE_FLAG;

  uint32_t um = 0, tk = 0;                     // per-step all-layer aggregates (App. E.2.6)
  trace_totals(s, 0, d.L, &um, &tk);
  s->hist_umiss.push_back(um);
  s->hist_tok_hits.push_back(tk);

  uint64_t resident_bytes = 0;
  rc = batched_waves(s, a, 0, d.L, &resident_bytes, op_res);
  if (rc != REMOE_OK) return rc;
  if (s->profiling) s->ev_used[prof_slot].bytes = resident_bytes;
  CK(launch_combine_batched(a, hout, 0, d.L, nullptr, s->stream));
  s->kernel_launches += 1;
  l_op(s, kStCompute);
  return l_verdict(s);
}

// Chained step for B > 1: every layer has its own norm -> route -> trace -> waves -> combine round trip,
// the B sequences moving through the layers together (they share each layer's cache).
int decode_step_chained_batched(remoe_stack* s, const float* hin, float* hout, float* layer_inputs, int32_t* ids,
                                float* gates) {
  DevStack& d = s->d;
  d.has_prev = s->steps_since_reset > 0 ? 1 : 0;
  d.policy = s->policy;
  d.beta = s->beta;
  const size_t rows = (size_t)d.B * d.H;
  CK(cudaMemcpyAsync(s->chain_in, hin, rows * sizeof(float), cudaMemcpyDeviceToDevice, s->stream));

  BatchArgs a{};
  a.d = d;
  a.hidden_in = s->chain_x;
  a.gates = gates;
  a.part = s->part;
  a.flags = s->flags;
  a.plan = s->plan;
  a.max_items = s->max_items;
  a.step_id = ++s->step_serial;
  uint32_t um = 0, tk = 0;
  for (int l = 0; l < d.L; ++l) {
    CK(launch_rmsnorm(s->chain_in + l * rows, s->chain_x + l * rows, d.H, d.B, s->stream));
    CK(launch_route(d, s->chain_x, ids, gates, s->contrib, l, 1, s->stream));
    s->kernel_launches += 3;
    l_op(s, kStCompute);
    CK(cudaEventRecord(s->ev_trace, s->stream));
    l_record(s, s->ev_trace, kStCompute);
    a.phase = 0;
    a.layer = l;
    a.depth = 0;
    CK(launch_batched(s, a));
    s->kernel_launches += 2;
    const LOp op_res = l_op(s, kStCompute);
    CK(cudaEventRecord(s->ev_resident, s->stream));
    l_record(s, s->ev_resident, kStCompute);
    CK(cudaEventSynchronize(s->ev_trace));
    l_host_wait(s, s->ev_trace);
    if (check_device_flag(s) != REMOE_OK) return REMOE_E_DEVICE_FLAG;
    trace_totals(s, l, l + 1, &um, &tk);
    uint64_t unused = 0;
    int rc = batched_waves(s, a, l, l + 1, &unused, op_res);
    if (rc != REMOE_OK) return rc;
    CK(launch_combine_batched(a, s->chain_out, l, 1, s->chain_in, s->stream));
    s->kernel_launches += 1;
    l_op(s, kStCompute);
  }
  s->steps += 1;
  s->steps_since_reset += 1;
  s->hist_umiss.push_back(um);
  s->hist_tok_hits.push_back(tk);
  CK(cudaMemcpyAsync(hout, s->chain_in + d.L * rows, rows * sizeof(float), cudaMemcpyDeviceToDevice, s->stream));
  if (layer_inputs)
    CK(cudaMemcpyAsync(layer_inputs, s->chain_in, rows * d.L * sizeof(float), cudaMemcpyDeviceToDevice,
                       s->stream));
  return l_verdict(s);
}

}  // namespace

extern "C" {

const char* remoe_strerror(int code) {
  switch (code) {
    case REMOE_OK: return "ok";
    case REMOE_E_ARG: return "invalid argument";
    case REMOE_E_CAPACITY: return "cache capacity below top_k";
    case REMOE_E_NOT_LOADED: return "weights not loaded";
    case REMOE_E_NOT_PINNED: return "expert pointer is not page-locked host memory";
    case REMOE_E_CUDA: return "CUDA runtime error";
    case REMOE_E_DEVICE_FLAG: return "device-side error flag set";
    case REMOE_E_UNSUPPORTED: return "unsupported shape";
    case REMOE_E_NOMEM: return "out of memory";
    case REMOE_E_ORDER: return "schedule ordering check failed";
    default: return "unknown error";
  }
}

const char* remoe_last_cuda_error(const remoe_stack* s) { return s ? s->cuda_err.c_str() : ""; }

void remoe_stack_destroy(remoe_stack* s) {
  if (!s) return;
  DeviceGuard guard(s->device);
  cudaStreamSynchronize(s->stream);
  if (s->copy_stream) {
    cudaStreamSynchronize(s->copy_stream);
    cudaStreamDestroy(s->copy_stream);
  }
  for (EvPair& p : s->ev_used) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  for (EvPair& p : s->ev_free) { cudaEventDestroy(p.a); cudaEventDestroy(p.b); }
  if (s->ev_trace) cudaEventDestroy(s->ev_trace);
  if (s->ev_resident) cudaEventDestroy(s->ev_resident);
  for (cudaEvent_t e : s->ev_stage) if (e) cudaEventDestroy(e);
  if (s->route_stream) {
    cudaStreamSynchronize(s->route_stream);
    cudaStreamDestroy(s->route_stream);
  }
  if (s->ev_entry) cudaEventDestroy(s->ev_entry);
  for (int p = 0; p < 2; ++p) {
    if (s->ev_route2[p]) cudaEventDestroy(s->ev_route2[p]);
    if (s->ev_free2[p]) cudaEventDestroy(s->ev_free2[p]);
    if (s->ev_res2[p]) cudaEventDestroy(s->ev_res2[p]);
  }
  for (cudaEvent_t e : s->ev_copy2) cudaEventDestroy(e);
  for (cudaEvent_t e : s->ev_miss2) cudaEventDestroy(e);
  for (cudaEvent_t e : s->ev_pool) cudaEventDestroy(e);
  for (cudaEvent_t e : s->ev_layer) cudaEventDestroy(e);
  for (void* p : s->dev_allocs) cudaFree(p);
  for (void* p : s->host_allocs) cudaFreeHost(p);
  delete s;
}

int remoe_stack_create(const remoe_shape* sh, int32_t cache_slots, void* cuda_stream, remoe_stack** out) {
  if (!sh || !out) return REMOE_E_ARG;
  *out = nullptr;
  if (sh->n_layers < 1 || sh->hidden < 1 || sh->n_routed < 1 || sh->top_k < 1 || sh->inter_routed < 1 ||
      sh->batch < 1 || sh->n_shared < 0 || cache_slots < 1 || sh->top_k > sh->n_routed ||
      (sh->n_shared > 0 && sh->inter_shared < 1) || (sh->weight_dtype != REMOE_F32 && sh->weight_dtype != REMOE_BF16 && sh->weight_dtype != REMOE_FP8_E4M3 &&
       sh->weight_dtype != REMOE_INT4_G32))
    return REMOE_E_ARG;
  if (sh->batch == 1 && cache_slots < sh->top_k) return REMOE_E_CAPACITY;
  // host store: bytes per element, 0 tagging the 4-bit grouped format
  const int wbytes = sh->weight_dtype == REMOE_BF16 ? 2
                     : sh->weight_dtype == REMOE_FP8_E4M3 ? 1 : sh->weight_dtype == REMOE_INT4_G32 ? 0 : 4;

  const int rbytes = sh->weight_dtype == REMOE_F32 ? 4 : 2;
  // A batched stack over an FP8 store keeps its slots as bf16 operand tiles: fetched bytes are widened on arrival.
  const bool widen = (sh->weight_dtype == REMOE_FP8_E4M3 || sh->weight_dtype == REMOE_INT4_G32) && sh->batch > 1;
  const int dev_wbytes = widen ? 2 : wbytes;
  const long pairs = (long)sh->n_layers * (sh->top_k + sh->n_shared);
  if (sh->hidden > kMaxHidden || sh->n_routed > kMaxRouted || sh->top_k > 32 || cache_slots > kMaxSlots || cache_slots > sh->n_routed ||
      (long)sh->batch * sh->top_k > kMaxRequests || !ffn_stream_supported(sh->hidden, wbytes))
    return REMOE_E_UNSUPPORTED;
  if (sh->batch == 1 && pairs > kMaxPairs) return REMOE_E_UNSUPPORTED;

  remoe_stack* s = new (std::nothrow) remoe_stack();
  if (!s) return REMOE_E_NOMEM;
  s->shape = *sh;
  s->C = cache_slots;
  s->stream = static_cast<cudaStream_t>(cuda_stream);
  s->BK = sh->batch * sh->top_k;
  int rc = REMOE_OK;
  auto bail = [&](int code) {
    remoe_stack_destroy(s);
    return code;
  };
  if (cudaGetDevice(&s->device) != cudaSuccess) return bail(REMOE_E_CUDA);
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, s->device) != cudaSuccess || sms < 1)
    return bail(REMOE_E_CUDA);
  s->grid = sms;
  if (cudaStreamCreateWithFlags(&s->copy_stream, cudaStreamNonBlocking) != cudaSuccess) return bail(REMOE_E_CUDA);
  if (cudaEventCreateWithFlags(&s->ev_trace, cudaEventDisableTiming) != cudaSuccess) return bail(REMOE_E_CUDA);
  s->ev_layer.resize(sh->n_layers, nullptr);
  for (auto& e : s->ev_layer)
    if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return bail(REMOE_E_CUDA);

  if (const char* chk = std::getenv("REMOE_CHECK_ORDER"))
    if (std::strcmp(chk, "1") == 0) s->ledger.reset(new (std::nothrow) OrderLedger());
  if (const char* inj = std::getenv("REMOE_FAULT_INJECT"))
    s->inject_lost_copy = std::strcmp(inj, "lost_copy") == 0 && sh->batch == 1;
  DevStack& d = s->d;
  d.L = sh->n_layers; d.H = sh->hidden; d.N = sh->n_routed; d.K = sh->top_k; d.I = sh->inter_routed;
  d.S = sh->n_shared; d.Is = sh->n_shared ? sh->inter_shared : 0; d.B = sh->batch; d.C = cache_slots;
  d.shared_gate = sh->shared_gate ? 1 : 0; d.renorm = sh->renorm_topk ? 1 : 0; d.wbytes = dev_wbytes; d.rbytes = rbytes;
  d.policy = REMOE_POLICY_LRU; d.beta = 0.f; d.has_prev = 0;
  d.slot_bytes = (size_t)3 * d.I * weight_row_bytes(d.H, dev_wbytes);
  d.shared_bytes = (size_t)3 * d.Is * weight_row_bytes(d.H, dev_wbytes);
  s->fetch_bytes = (size_t)3 * d.I * weight_row_bytes(d.H, wbytes);
  s->fetch_shared_bytes = (size_t)3 * d.Is * weight_row_bytes(d.H, wbytes);
  s->widen_fp8 = widen;
  s->host_wbytes = wbytes;
  const size_t L = d.L;
  char *router = nullptr, *sgw = nullptr, *shared = nullptr, *slots = nullptr;
#define TRY(x) do { rc = (x); if (rc != REMOE_OK) return bail(rc); } while (0)
  TRY(dev_alloc(s, &router, L * d.N * d.H * rbytes));
  TRY(dev_alloc(s, &sgw, L * d.H * rbytes));
  TRY(dev_alloc(s, &shared, L * d.S * d.shared_bytes));
  TRY(dev_alloc(s, &slots, L * d.C * d.slot_bytes));
  d.router = router; d.shared_gate_w = sgw; d.shared_blocks = shared; d.slots = slots;
  TRY(dev_alloc(s, &d.expert_of_slot, L * d.C));
  TRY(dev_alloc(s, &d.slot_of_expert, L * d.N));
  TRY(dev_alloc(s, &d.stamp, L * d.C));
  TRY(dev_alloc(s, &d.freq, L * d.C));
  TRY(dev_alloc(s, &d.clock, L));
  TRY(dev_alloc(s, &d.prev_mask, L * d.B * kMaskWords));
  TRY(dev_alloc(s, &d.counters, L * kCounters));
  TRY(dev_alloc(s, &d.load, L * d.N));
  TRY(dev_alloc(s, &d.shared_scale, L * d.B));
  TRY(dev_alloc(s, &d.last_overlap, L * d.B));
  TRY(dev_alloc(s, &d.last_mass, L * d.B));
  TRY(dev_alloc(s, &d.mass_sum, L * d.B));
  s->block_ints = 1 + (size_t)trace_ints(d.L, s->BK);
  TRY(dev_alloc(s, &s->dev_block, s->block_ints));
  TRY(host_alloc(s, &s->host_block, s->block_ints));
  std::memset(s->host_block, 0, s->block_ints * sizeof(int));
  d.err = s->dev_block;
  d.trace = s->dev_block + 1;
  {
    void* dp = nullptr;
    if (cudaHostGetDevicePointer(&dp, s->host_block, 0) != cudaSuccess || !dp) return bail(REMOE_E_CUDA);
    d.host_mirror = static_cast<int*>(dp);
  }
  TRY(dev_alloc(s, &s->partial, (size_t)2 * L * s->grid * d.H));
  TRY(dev_alloc(s, &s->contrib, (size_t)2 * L * 2));
  TRY(dev_alloc(s, &s->chain_in, (L + 1) * d.B * d.H));
  TRY(dev_alloc(s, &s->chain_out, L * d.B * d.H));
  TRY(dev_alloc(s, &s->chain_x, L * d.B * d.H));
  TRY(dev_alloc(s, &s->link_ticket, 1));
  if (cudaMemset(s->link_ticket, 0, sizeof(unsigned)) != cudaSuccess) return bail(REMOE_E_CUDA);
  if (d.B > 1) {
    if (!ffn_batched_supported(d)) return bail(REMOE_E_UNSUPPORTED);
    const size_t P = d.K + d.S;
    TRY(dev_alloc(s, &d.grp_count, L * s->BK));
    TRY(dev_alloc(s, &d.grp_tok, L * s->BK * d.B));
    TRY(dev_alloc(s, &d.grp_k, L * s->BK * d.B));
    TRY(dev_alloc(s, &s->part, L * d.B * P * kUnitsPerItem * d.H));
    TRY(dev_alloc(s, &s->flags, L * d.B * P * kUnitsPerItem));
    s->max_items = (int)(L * (s->BK + (size_t)d.S * ((d.B + kMinTokTile - 1) / kMinTokTile))) + 1;
    TRY(dev_alloc(s, &s->plan, (size_t)8 + 4 * (size_t)s->max_items));
    if (cudaMemset(s->flags, 0, L * d.B * P * kUnitsPerItem * sizeof(int)) != cudaSuccess) return bail(REMOE_E_CUDA);
    if (cudaEventCreateWithFlags(&s->ev_resident, cudaEventDisableTiming) != cudaSuccess) return bail(REMOE_E_CUDA);
    const char* pick = std::getenv("REMOE_BATCHED_KERNEL");      // "mma" forces the mma.sync kernel
    if (ffn_batched_tc_supported(d) && ffn_batched_tc_maps_bytes() <= sizeof(s->tc_maps) &&
        !(pick && std::strcmp(pick, "mma") == 0)) {
      s->stage_bytes = std::max((size_t)2 * d.C * s->fetch_bytes, s->fetch_shared_bytes);
      TRY(dev_alloc(s, &s->stage_pool, s->stage_bytes));
      for (cudaEvent_t& e : s->ev_stage)
        if (cudaEventCreateWithFlags(&e, cudaEventDisableTiming) != cudaSuccess) return bail(REMOE_E_CUDA);
      // (the tensor maps describe a bf16 staging pool; FP8 blocks are rewritten by the widening kernel instead)
      if (!widen && ffn_batched_tc_init(d, s->stage_pool, s->stage_bytes, s->tc_maps) != cudaSuccess)
        return bail(REMOE_E_CUDA);
      s->use_tc = true;
    }
    if (widen && !s->use_tc) return bail(REMOE_E_UNSUPPORTED);
  }
  const size_t io = L * d.B * d.H, kk = L * (size_t)s->BK;
  TRY(dev_alloc(s, &s->st_in_d, io));
  TRY(dev_alloc(s, &s->st_out_d, io));
  TRY(dev_alloc(s, &s->st_g_d, kk));
  TRY(dev_alloc(s, &s->st_ids_d, kk));
  TRY(host_alloc(s, &s->st_in_h, io));
  TRY(host_alloc(s, &s->st_out_h, io));
  TRY(host_alloc(s, &s->st_g_h, kk));
  TRY(host_alloc(s, &s->st_ids_h, kk));
#undef TRY
  s->host_ptrs.assign(L * d.N, nullptr);
  s->router_loaded.assign(L, 0);
  s->shared_loaded.assign(L * d.S, 0);
  s->h2d_bytes.assign(L, 0);
  rc = reset_state(s);
  if (rc != REMOE_OK) return bail(rc);
  *out = s;
  return REMOE_OK;
}

int remoe_load_router(remoe_stack* s, int32_t layer, const void* w, const void* wsg) {
  if (!s || !w || layer < 0 || layer >= s->d.L) return REMOE_E_ARG;
  if (s->d.shared_gate && !wsg) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  const size_t row = (size_t)s->d.H * s->d.rbytes;
  CK(cudaMemcpyAsync(const_cast<char*>(s->d.router) + (size_t)layer * s->d.N * row, w, s->d.N * row,
                     cudaMemcpyHostToDevice, s->stream));
  if (s->d.shared_gate)
    CK(cudaMemcpyAsync(const_cast<char*>(s->d.shared_gate_w) + (size_t)layer * row, wsg, row,
                       cudaMemcpyHostToDevice, s->stream));
  CK(cudaStreamSynchronize(s->stream));
  s->router_loaded[layer] = 1;
  return REMOE_OK;
}

int remoe_load_shared(remoe_stack* s, int32_t layer, int32_t idx, const void* block) {
  if (!s || !block || layer < 0 || layer >= s->d.L || idx < 0 || idx >= s->d.S) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  char* dst = const_cast<char*>(s->d.shared_blocks) + ((size_t)layer * s->d.S + idx) * s->d.shared_bytes;
  if (s->use_tc) {
    // such a stack keeps its blocks in operand-tile order: land in the staging pool, then retile
    CK(cudaStreamSynchronize(s->copy_stream));
    CK(cudaStreamSynchronize(s->stream));
    CK(cudaMemcpyAsync(s->stage_pool, block, s->fetch_shared_bytes, cudaMemcpyHostToDevice, s->stream));
    const size_t off = 0;
    if (s->widen_fp8) {
      const void* src = s->stage_pool;
      CK(launch_widen_retile_tc(s->d, s->host_wbytes, 1, &src, &dst, s->d.Is, s->stream));
    } else {
      CK(launch_retile_tc(s->d, s->tc_maps, 1, &off, &dst, s->d.Is, s->stream));
    }
    s->kernel_launches += 1;
  } else {
    CK(cudaMemcpyAsync(dst, block, s->d.shared_bytes, cudaMemcpyHostToDevice, s->stream));
  }
  CK(cudaStreamSynchronize(s->stream));
  s->shared_loaded[(size_t)layer * s->d.S + idx] = 1;
  return REMOE_OK;
}

int remoe_load_experts_host(remoe_stack* s, int32_t layer, int32_t first, int32_t count,
                            const void* const* ptrs) {
  if (!s || !ptrs || layer < 0 || layer >= s->d.L || first < 0 || count < 0 || first + count > s->d.N)
    return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  for (int i = 0; i < count; ++i) {
    if (!ptrs[i] || (reinterpret_cast<uintptr_t>(ptrs[i]) & 15u)) return REMOE_E_ARG;
    cudaPointerAttributes at{};
    cudaError_t e = cudaPointerGetAttributes(&at, ptrs[i]);
    if (e != cudaSuccess) {
      cudaGetLastError();
      return REMOE_E_NOT_PINNED;
    }
    if (at.type != cudaMemoryTypeHost) return REMOE_E_NOT_PINNED;
  }
  for (int i = 0; i < count; ++i) s->host_ptrs[(size_t)layer * s->d.N + first + i] = ptrs[i];
  return REMOE_OK;
}

int remoe_decode_step(remoe_stack* s, const float* hin, float* hout, int32_t* ids, float* gates) {
  if (!s || !hin || !hout || !ids || !gates) return REMOE_E_ARG;
  if ((reinterpret_cast<uintptr_t>(hin) | reinterpret_cast<uintptr_t>(hout)) & 15u) return REMOE_E_ARG;
  if (!everything_loaded(s)) return REMOE_E_NOT_LOADED;
  ON_STACK_DEVICE(s);
  if (s->d.B != 1) return decode_step_batched(s, hin, hout, ids, gates);
  DevStack& d = s->d;
  d.has_prev = s->steps_since_reset > 0 ? 1 : 0;
  d.policy = s->policy;
  d.beta = s->beta;

  CK(launch_route(d, hin, ids, gates, s->contrib, 0, d.L, s->stream));
  s->kernel_launches += d.B > 1 ? 2 : 1;
  l_op(s, kStCompute);
  CK(cudaEventRecord(s->ev_trace, s->stream));      // the route kernel has written the trace to the host mirror
  l_record(s, s->ev_trace, kStCompute);

  FfnArgs a{};
  a.d = d;
  a.hidden_in = hin;
  a.gates = gates;
  a.partial = s->partial;
  a.contrib = s->contrib;
  a.grid_cap = s->grid;
  a.phase = 0;
  a.layer = -1;
  // The resident phase needs no host decision: enqueue it before waiting for the trace.
  int rc = prof_begin(s, s->stream, 0, 0);
  if (rc != REMOE_OK) return rc;
  if (s->inject_lost_copy) {
    a.lose_row1 = 1;                 // the launch's first weight row never arrives
    a.spin_limit = 1u << 12;         // so that the wait for it gives up quickly
    s->inject_lost_copy = false;
  }
  CK(launch_ffn_stream(a, s->grid, s->stream));
  a.lose_row1 = 0;
  a.spin_limit = 0;
  s->kernel_launches += 1;
  const LOp op_res = l_op(s, kStCompute);
  rc = prof_end(s, s->stream);
  if (rc != REMOE_OK) return rc;
  const size_t prof_slot = s->profiling ? s->ev_used.size() - 1 : 0;

  CK(cudaEventSynchronize(s->ev_trace));
  l_host_wait(s, s->ev_trace);
  s->steps += 1;
  s->steps_since_reset += 1;
  if (check_device_flag(s) != REMOE_OK) return REMOE_E_DEVICE_FLAG;

  {
    uint32_t um = 0, tk = 0;                   // per-step all-layer aggregates (App. E.2.6)
    trace_totals(s, 0, d.L, &um, &tk);
    s->hist_umiss.push_back(um);
    s->hist_tok_hits.push_back(tk);
  }

  int* tr = s->host_block + 1;
  const int* t_req = trace_requests(tr, d.L, s->BK);
  const int* t_hit = trace_hit(tr, d.L, s->BK);
  const int* t_slot = trace_slot(tr, d.L, s->BK);
  uint64_t resident_bytes = 0;
  bool copy_ordered = false;
  for (int l = 0; l < d.L; ++l) {
    int misses = 0;
    for (int k = 0; k < d.K; ++k) {
      const int i = l * s->BK + k;
      if (t_hit[i]) {
        resident_bytes += d.slot_bytes;
        if (t_slot[i] >= 0 && t_slot[i] < d.C) l_read(s, op_res, slot_cell(s, l, t_slot[i]), "resident-phase launch");
        continue;
      }
      const int e = t_req[i], slot = t_slot[i];
      if (e < 0 || e >= d.N || slot < 0 || slot >= d.C) {
        s->cuda_err = "trace holds an expert id or slot out of range (layer " + std::to_string(l) + ")";
        return REMOE_E_DEVICE_FLAG;
      }
      if (!copy_ordered) {
        // Victim slots may still be read by the previous step's kernels, all of which precede
        // this step's route kernel on the compute stream.
        CK(cudaStreamWaitEvent(s->copy_stream, s->ev_trace, 0));
        l_wait(s, kStCopy, s->ev_trace);
        copy_ordered = true;
      }
      CK(cudaMemcpyAsync(d.slots + ((size_t)l * d.C + slot) * d.slot_bytes, s->host_ptrs[(size_t)l * d.N + e],
                         d.slot_bytes, cudaMemcpyHostToDevice, s->copy_stream));
      l_write(s, l_op(s, kStCopy), slot_cell(s, l, slot), "miss fetch");
      ++misses;
    }
    resident_bytes += (uint64_t)d.S * d.shared_bytes;
    if (misses) {
      s->h2d_bytes[l] += (uint64_t)misses * d.slot_bytes;
      CK(cudaEventRecord(s->ev_layer[l], s->copy_stream));
      l_record(s, s->ev_layer[l], kStCopy);
      CK(cudaStreamWaitEvent(s->stream, s->ev_layer[l], 0));
      l_wait(s, kStCompute, s->ev_layer[l]);
      a.phase = 1;
      a.layer = l;
      rc = prof_begin(s, s->stream, (uint64_t)misses * d.slot_bytes, 1);
      if (rc != REMOE_OK) return rc;
      CK(launch_ffn_stream(a, s->grid, s->stream));
      s->kernel_launches += 1;
      if (s->ledger) {
        const LOp om = l_op(s, kStCompute);
        for (int k = 0; k < d.K; ++k)
          if (!t_hit[l * s->BK + k]) l_read(s, om, slot_cell(s, l, t_slot[l * s->BK + k]), "miss-phase launch");
      }
      rc = prof_end(s, s->stream);
      if (rc != REMOE_OK) return rc;
    }
  }
  if (s->profiling) s->ev_used[prof_slot].bytes = resident_bytes;
  CK(launch_combine(a, hout, 0, d.L, nullptr, s->stream));
  s->kernel_launches += 1;
  l_op(s, kStCompute);
  return l_verdict(s);
}

// Second buffer set, route stream and events of remoe_decode_steps.
static int pipe_setup(remoe_stack* s) {
  if (s->pipe_ready) return REMOE_OK;
  const DevStack& d = s->d;
  int rc;
  if ((rc = dev_alloc(s, &s->dev_block2, s->block_ints)) != REMOE_OK) return rc;
  if ((rc = host_alloc(s, &s->host_block2, s->block_ints)) != REMOE_OK) return rc;
  if ((rc = dev_alloc(s, &s->contrib2, (size_t)2 * d.L * 2)) != REMOE_OK) return rc;
  if ((rc = dev_alloc(s, &s->shared_scale2, (size_t)d.L * d.B)) != REMOE_OK) return rc;
  std::memset(s->host_block2, 0, s->block_ints * sizeof(int));
  CK(cudaMemset(s->dev_block2, 0, s->block_ints * sizeof(int)));
  if (!s->route_stream) CK(cudaStreamCreateWithFlags(&s->route_stream, cudaStreamNonBlocking));
  auto make = [&](cudaEvent_t* e) { return *e ? cudaSuccess : cudaEventCreateWithFlags(e, cudaEventDisableTiming); };
  CK(make(&s->ev_entry));
  for (int p = 0; p < 2; ++p) {
    CK(make(&s->ev_route2[p]));
    CK(make(&s->ev_free2[p]));
    CK(make(&s->ev_res2[p]));
  }
  s->ev_copy2.resize((size_t)2 * d.L, nullptr);
  s->ev_miss2.resize((size_t)2 * d.L, nullptr);
  for (auto& e : s->ev_copy2) CK(make(&e));
  for (auto& e : s->ev_miss2) CK(make(&e));
  s->pipe_ready = true;
  return REMOE_OK;
}

int remoe_decode_steps(remoe_stack* s, int32_t n_steps, const float* hin, float* hout, int32_t* ids, float* gates) {
  if (!s || !hin || !hout || !ids || !gates || n_steps < 0) return REMOE_E_ARG;
  if ((reinterpret_cast<uintptr_t>(hin) | reinterpret_cast<uintptr_t>(hout)) & 15u) return REMOE_E_ARG;
  if (!everything_loaded(s)) return REMOE_E_NOT_LOADED;
  if (s->d.B != 1) return REMOE_E_UNSUPPORTED;
  if (n_steps == 0) return REMOE_OK;
  ON_STACK_DEVICE(s);
  int rc = pipe_setup(s);
  if (rc != REMOE_OK) return rc;
  DevStack base = s->d;
  base.policy = s->policy;
  base.beta = s->beta;
  const int L = base.L, K = base.K;
  const size_t io = (size_t)L * base.H, kk = (size_t)L * K;

  // Step t uses buffer set t & 1 (device trace + host mirror, contributor table, shared scales).  Its
  // route kernel runs on the route stream as soon as the set is free (combine of step t-2) -- while
  // step t-1 is still fetching and computing -- so the host has the next miss list before the copy
  // engine runs dry.  A copy of step t into layer l waits for the kernels of step t-1 that read layer
  // l's slots: its resident-phase launch and, if it had misses there, that miss-phase launch.
  int* dev_blk[2] = {s->dev_block, s->dev_block2};
  int* host_blk[2] = {s->host_block, s->host_block2};
  int* contrib[2] = {s->contrib, s->contrib2};
  float* scale[2] = {s->d.shared_scale, s->shared_scale2};
  std::vector<char> missed[2] = {std::vector<char>(L, 0), std::vector<char>(L, 0)};

  CK(cudaEventRecord(s->ev_entry, s->stream));          // everything before the call, the inputs included
  CK(cudaStreamWaitEvent(s->route_stream, s->ev_entry, 0));
  CK(cudaStreamWaitEvent(s->copy_stream, s->ev_entry, 0));
  l_record(s, s->ev_entry, kStCompute);
  l_wait(s, kStRoute, s->ev_entry);
  l_wait(s, kStCopy, s->ev_entry);

  auto route = [&](int t) -> int {
    const int p = t & 1;
    DevStack d = base;
    d.has_prev = (s->steps_since_reset + (uint64_t)t) > 0 ? 1 : 0;
    d.trace = dev_blk[p] + 1;
    d.host_mirror = host_blk[p];
    d.shared_scale = scale[p];
    if (t >= 2) {
      CK(cudaStreamWaitEvent(s->route_stream, s->ev_free2[p], 0));
      l_wait(s, kStRoute, s->ev_free2[p]);
    }
    CK(launch_route(d, hin + (size_t)t * io, ids + (size_t)t * kk, gates + (size_t)t * kk, contrib[p], 0, L,
                    s->route_stream));
    s->kernel_launches += 1;
    l_op(s, kStRoute);
    CK(cudaEventRecord(s->ev_route2[p], s->route_stream));
    l_record(s, s->ev_route2[p], kStRoute);
    return REMOE_OK;
  };

  if ((rc = route(0)) != REMOE_OK) return rc;
  for (int t = 0; t < n_steps; ++t) {
    const int p = t & 1, q = p ^ 1;
    DevStack d = base;
    d.trace = dev_blk[p] + 1;
    d.host_mirror = host_blk[p];
    d.shared_scale = scale[p];
    FfnArgs a{};
    a.d = d;
    a.hidden_in = hin + (size_t)t * io;
    a.gates = gates + (size_t)t * kk;
    a.partial = s->partial;
    a.contrib = contrib[p];
    a.grid_cap = s->grid;
    a.phase = 0;
    a.layer = -1;
    CK(cudaStreamWaitEvent(s->stream, s->ev_route2[p], 0));
    l_wait(s, kStCompute, s->ev_route2[p]);
    rc = prof_begin(s, s->stream, 0, 0);
    if (rc != REMOE_OK) return rc;
    CK(launch_ffn_stream(a, s->grid, s->stream));
    s->kernel_launches += 1;
    const LOp op_res = l_op(s, kStCompute);
    rc = prof_end(s, s->stream);
    if (rc != REMOE_OK) return rc;
    const size_t prof_slot = s->profiling ? s->ev_used.size() - 1 : 0;
    CK(cudaEventRecord(s->ev_res2[p], s->stream));
    l_record(s, s->ev_res2[p], kStCompute);

    CK(cudaEventSynchronize(s->ev_route2[p]));
    l_host_wait(s, s->ev_route2[p]);
    s->steps += 1;
    if (check_device_flag(s, host_blk[p]) != REMOE_OK) {
      s->steps_since_reset += (uint64_t)t + 1;
      return REMOE_E_DEVICE_FLAG;
    }
    // the next step's routing needs nothing from this step's fetches or compute
    if (t + 1 < n_steps && (rc = route(t + 1)) != REMOE_OK) return rc;

    int* tr = host_blk[p] + 1;
    const int* t_req = trace_requests(tr, L, K);
    const int* t_hit = trace_hit(tr, L, K);
    const int* t_slot = trace_slot(tr, L, K);
    const int* t_th = trace_tok_hits(tr, L, K);
    uint32_t um = 0, tk = 0;
    uint64_t resident_bytes = 0;
    for (int l = 0; l < L; ++l) {
      int misses = 0;
      tk += (uint32_t)t_th[l];
      for (int k = 0; k < K; ++k) {
        const int i = l * K + k;
        if (t_hit[i]) {
          resident_bytes += d.slot_bytes;
          if (t_slot[i] >= 0 && t_slot[i] < d.C) l_read(s, op_res, slot_cell(s, l, t_slot[i]), "resident-phase launch");
          continue;
        }
        const int e = t_req[i], slot = t_slot[i];
        if (e < 0 || e >= d.N || slot < 0 || slot >= d.C) {
          s->cuda_err = "trace holds an expert id or slot out of range (layer " + std::to_string(l) + ")";
          s->steps_since_reset += (uint64_t)t + 1;
          return REMOE_E_DEVICE_FLAG;
        }
        if (!misses && t > 0) {
          CK(cudaStreamWaitEvent(s->copy_stream, s->ev_res2[q], 0));
          l_wait(s, kStCopy, s->ev_res2[q]);
          if (missed[q][l]) {
            CK(cudaStreamWaitEvent(s->copy_stream, s->ev_miss2[(size_t)q * L + l], 0));
            l_wait(s, kStCopy, s->ev_miss2[(size_t)q * L + l]);
          }
        }
        CK(cudaMemcpyAsync(d.slots + ((size_t)l * d.C + slot) * d.slot_bytes, s->host_ptrs[(size_t)l * d.N + e],
                           d.slot_bytes, cudaMemcpyHostToDevice, s->copy_stream));
        l_write(s, l_op(s, kStCopy), slot_cell(s, l, slot), "miss fetch");
        ++misses;
      }
      resident_bytes += (uint64_t)d.S * d.shared_bytes;
      missed[p][l] = misses ? 1 : 0;
      um += (uint32_t)misses;
      if (!misses) continue;
      s->h2d_bytes[l] += (uint64_t)misses * d.slot_bytes;
      CK(cudaEventRecord(s->ev_copy2[(size_t)p * L + l], s->copy_stream));
      l_record(s, s->ev_copy2[(size_t)p * L + l], kStCopy);
      CK(cudaStreamWaitEvent(s->stream, s->ev_copy2[(size_t)p * L + l], 0));
      l_wait(s, kStCompute, s->ev_copy2[(size_t)p * L + l]);
      a.phase = 1;
      a.layer = l;
      rc = prof_begin(s, s->stream, (uint64_t)misses * d.slot_bytes, 1);
      if (rc != REMOE_OK) return rc;
      CK(launch_ffn_stream(a, s->grid, s->stream));
      s->kernel_launches += 1;
      if (s->ledger) {
        const LOp om = l_op(s, kStCompute);
        for (int k = 0; k < K; ++k)
          if (!t_hit[l * K + k]) l_read(s, om, slot_cell(s, l, t_slot[l * K + k]), "miss-phase launch");
      }
      rc = prof_end(s, s->stream);
      if (rc != REMOE_OK) return rc;
      CK(cudaEventRecord(s->ev_miss2[(size_t)p * L + l], s->stream));
      l_record(s, s->ev_miss2[(size_t)p * L + l], kStCompute);
    }
    if (s->profiling) s->ev_used[prof_slot].bytes = resident_bytes;
    s->hist_umiss.push_back(um);
    s->hist_tok_hits.push_back(tk);
    CK(launch_combine(a, hout + (size_t)t * io, 0, L, nullptr, s->stream));
    s->kernel_launches += 1;
    l_op(s, kStCompute);
    CK(cudaEventRecord(s->ev_free2[p], s->stream));
    l_record(s, s->ev_free2[p], kStCompute);
  }
  s->steps_since_reset += (uint64_t)n_steps;
  // Later calls use buffer set 0 and the stack's stream: leave the copy stream behind this call's last
  // readers, and the device trace of the last step where remoe_last_step_trace looks for it.
  CK(cudaStreamWaitEvent(s->copy_stream, s->ev_free2[(n_steps - 1) & 1], 0));
  l_wait(s, kStCopy, s->ev_free2[(n_steps - 1) & 1]);
  if ((n_steps - 1) & 1) {
    CK(cudaMemcpyAsync(s->dev_block + 1, s->dev_block2 + 1, (s->block_ints - 1) * sizeof(int),
                       cudaMemcpyDeviceToDevice, s->stream));
    CK(cudaMemcpyAsync(s->d.shared_scale, s->shared_scale2, (size_t)L * base.B * sizeof(float),
                       cudaMemcpyDeviceToDevice, s->stream));
  }
  return l_verdict(s);
}

int remoe_decode_step_chained(remoe_stack* s, const float* hin, float* hout, float* layer_inputs, int32_t* ids,
                              float* gates) {
  if (!s || !hin || !hout || !ids || !gates) return REMOE_E_ARG;
  if (!everything_loaded(s)) return REMOE_E_NOT_LOADED;
  ON_STACK_DEVICE(s);
  if (s->d.B != 1) return decode_step_chained_batched(s, hin, hout, layer_inputs, ids, gates);
  DevStack& d = s->d;
  d.has_prev = s->steps_since_reset > 0 ? 1 : 0;
  d.policy = s->policy;
  d.beta = s->beta;
  const size_t row = (size_t)d.H * sizeof(float);
  CK(cudaMemcpyAsync(s->chain_in, hin, row, cudaMemcpyDeviceToDevice, s->stream));

  FfnArgs a{};
  a.d = d;
  a.hidden_in = s->chain_x;
  a.gates = gates;
  a.partial = s->partial;
  a.contrib = s->contrib;
  a.grid_cap = s->grid;
  uint32_t um = 0, tk = 0;
  // The layer's input exists only once the previous layer is done, so every layer has its own
  // norm -> route -> trace -> fetch -> compute round trip.  The link kernel joins two layers in one
  // launch: sum of the upper layer's partials, residual add, pre-norm and routing of the lower layer.
  CK(launch_chain_link(d, a, 0, s->chain_in, s->chain_out, s->chain_x, s->link_ticket, 0, 1, ids, gates, s->stream));
  s->kernel_launches += 1;
  for (int l = 0; l < d.L; ++l) {
    l_op(s, kStCompute);
    CK(cudaEventRecord(s->ev_trace, s->stream));
    l_record(s, s->ev_trace, kStCompute);
    a.phase = 0;
    a.layer = l;
    CK(launch_ffn_stream(a, s->grid, s->stream));
    s->kernel_launches += 1;
    const LOp op_res = l_op(s, kStCompute);
    CK(cudaEventSynchronize(s->ev_trace));
    l_host_wait(s, s->ev_trace);
    if (check_device_flag(s) != REMOE_OK) return REMOE_E_DEVICE_FLAG;
    int* tr = s->host_block + 1;
    const int* t_req = trace_requests(tr, d.L, s->BK);
    const int* t_hit = trace_hit(tr, d.L, s->BK);
    const int* t_slot = trace_slot(tr, d.L, s->BK);
    tk += (uint32_t)trace_tok_hits(tr, d.L, s->BK)[l];
    int misses = 0;
    for (int k = 0; k < d.K; ++k) {
      const int i = l * s->BK + k;
      if (t_hit[i]) {
        if (t_slot[i] >= 0 && t_slot[i] < d.C) l_read(s, op_res, slot_cell(s, l, t_slot[i]), "resident-phase launch");
        continue;
      }
      const int e = t_req[i], slot = t_slot[i];
      if (e < 0 || e >= d.N || slot < 0 || slot >= d.C) {
        s->cuda_err = "trace holds an expert id or slot out of range (layer " + std::to_string(l) + ")";
        return REMOE_E_DEVICE_FLAG;
      }
      if (!misses) {
        CK(cudaStreamWaitEvent(s->copy_stream, s->ev_trace, 0));
        l_wait(s, kStCopy, s->ev_trace);
      }
      CK(cudaMemcpyAsync(d.slots + ((size_t)l * d.C + slot) * d.slot_bytes, s->host_ptrs[(size_t)l * d.N + e],
                         d.slot_bytes, cudaMemcpyHostToDevice, s->copy_stream));
      l_write(s, l_op(s, kStCopy), slot_cell(s, l, slot), "miss fetch");
      ++misses;
    }
    um += (uint32_t)misses;
    if (misses) {
      s->h2d_bytes[l] += (uint64_t)misses * d.slot_bytes;
      CK(cudaEventRecord(s->ev_layer[l], s->copy_stream));
      l_record(s, s->ev_layer[l], kStCopy);
      CK(cudaStreamWaitEvent(s->stream, s->ev_layer[l], 0));
      l_wait(s, kStCompute, s->ev_layer[l]);
      a.phase = 1;
      CK(launch_ffn_stream(a, s->grid, s->stream));
      s->kernel_launches += 1;
      if (s->ledger) {
        const LOp om = l_op(s, kStCompute);
        for (int k = 0; k < d.K; ++k)
          if (!t_hit[l * s->BK + k]) l_read(s, om, slot_cell(s, l, t_slot[l * s->BK + k]), "miss-phase launch");
      }
    }
    // the link also reads the contributor table the miss-phase launch (if any) has just completed
    CK(launch_chain_link(d, a, l + 1, s->chain_in, s->chain_out, s->chain_x, s->link_ticket, 1, l + 1 < d.L ? 1 : 0, ids,
                         gates, s->stream));
    s->kernel_launches += 1;
  }
  l_op(s, kStCompute);
  s->steps += 1;
  s->steps_since_reset += 1;
  s->hist_umiss.push_back(um);
  s->hist_tok_hits.push_back(tk);
  CK(cudaMemcpyAsync(hout, s->chain_in + (size_t)d.L * d.H, row, cudaMemcpyDeviceToDevice, s->stream));
  if (layer_inputs)
    CK(cudaMemcpyAsync(layer_inputs, s->chain_in, row * d.L, cudaMemcpyDeviceToDevice, s->stream));
  return l_verdict(s);
}

int remoe_decode_step_host(remoe_stack* s, const float* hin, float* hout, int32_t* ids, float* gates) {
  if (!s || !hin || !hout || !ids || !gates) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  const size_t io = (size_t)s->d.L * s->d.B * s->d.H, kk = (size_t)s->d.L * s->BK;
  std::memcpy(s->st_in_h, hin, io * sizeof(float));
  CK(cudaMemcpyAsync(s->st_in_d, s->st_in_h, io * sizeof(float), cudaMemcpyHostToDevice, s->stream));
  int rc = remoe_decode_step(s, s->st_in_d, s->st_out_d, s->st_ids_d, s->st_g_d);
  if (rc != REMOE_OK) return rc;
  CK(cudaMemcpyAsync(s->st_out_h, s->st_out_d, io * sizeof(float), cudaMemcpyDeviceToHost, s->stream));
  CK(cudaMemcpyAsync(s->st_ids_h, s->st_ids_d, kk * sizeof(int), cudaMemcpyDeviceToHost, s->stream));
  CK(cudaMemcpyAsync(s->st_g_h, s->st_g_d, kk * sizeof(float), cudaMemcpyDeviceToHost, s->stream));
  CK(cudaStreamSynchronize(s->stream));
  rc = fetch_device_flag(s);                   // an expert kernel of this very step may have given up
  if (rc != REMOE_OK) return rc;
  std::memcpy(hout, s->st_out_h, io * sizeof(float));
  std::memcpy(ids, s->st_ids_h, kk * sizeof(int));
  std::memcpy(gates, s->st_g_h, kk * sizeof(float));
  return REMOE_OK;
}

int remoe_last_step_trace(remoe_stack* s, int32_t* req, int32_t* hit, int32_t* slot, int32_t* ev, int32_t* nu) {
  if (!s) return REMOE_E_ARG;
  if (s->steps == 0) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  CK(cudaMemcpy(s->host_block, s->dev_block, s->block_ints * sizeof(int), cudaMemcpyDeviceToHost));
  int* tr = s->host_block + 1;
  const size_t n = (size_t)s->d.L * s->BK * sizeof(int);
  if (req) std::memcpy(req, trace_requests(tr, s->d.L, s->BK), n);
  if (hit) std::memcpy(hit, trace_hit(tr, s->d.L, s->BK), n);
  if (slot) std::memcpy(slot, trace_slot(tr, s->d.L, s->BK), n);
  if (ev) std::memcpy(ev, trace_evicted(tr, s->d.L, s->BK), n);
  if (nu) std::memcpy(nu, trace_n_unique(tr), (size_t)s->d.L * sizeof(int));
  return check_device_flag(s);
}

int remoe_cache_snapshot(remoe_stack* s, int32_t layer, int32_t* eos, uint64_t* stamp, uint32_t* use_count) {
  if (!s || layer < 0 || layer >= s->d.L) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  const size_t C = s->d.C, off = (size_t)layer * C;
  if (eos) CK(cudaMemcpy(eos, s->d.expert_of_slot + off, C * sizeof(int), cudaMemcpyDeviceToHost));
  if (stamp) CK(cudaMemcpy(stamp, s->d.stamp + off, C * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  if (use_count) CK(cudaMemcpy(use_count, s->d.freq + off, C * sizeof(unsigned), cudaMemcpyDeviceToHost));
  return fetch_device_flag(s);
}

int remoe_cache_stats(remoe_stack* s, int32_t layer, remoe_cache_counters* out) {
  if (!s || !out || layer < -1 || layer >= s->d.L) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  std::vector<unsigned long long> c((size_t)s->d.L * kCounters);
  CK(cudaMemcpy(c.data(), s->d.counters, c.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  std::memset(out, 0, sizeof(*out));
  for (int l = 0; l < s->d.L; ++l) {
    if (layer >= 0 && l != layer) continue;
    out->tok_hits += c[(size_t)l * kCounters + 0];
    out->tok_misses += c[(size_t)l * kCounters + 1];
    out->uniq_hits += c[(size_t)l * kCounters + 2];
    out->uniq_misses += c[(size_t)l * kCounters + 3];
    out->h2d_bytes += s->h2d_bytes[l];
  }
  out->steps = s->steps;
  return fetch_device_flag(s);
}

int remoe_reuse_stats(remoe_stack* s, int32_t layer, uint64_t* overlap_sum, uint64_t* pairs, float* last_ir) {
  if (!s || layer < -1 || layer >= s->d.L) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  std::vector<unsigned long long> c((size_t)s->d.L * kCounters);
  CK(cudaMemcpy(c.data(), s->d.counters, c.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  uint64_t o = 0, p = 0;
  for (int l = 0; l < s->d.L; ++l) {
    if (layer >= 0 && l != layer) continue;
    o += c[(size_t)l * kCounters + 4];
    p += c[(size_t)l * kCounters + 5];
  }
  if (overlap_sum) *overlap_sum = o;
  if (pairs) *pairs = p;
  if (last_ir) {
    std::vector<int> ov((size_t)s->d.L * s->d.B);
    CK(cudaMemcpy(ov.data(), s->d.last_overlap, ov.size() * sizeof(int), cudaMemcpyDeviceToHost));
    const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? s->d.L : layer + 1;
    size_t j = 0;
    for (int l = l0; l < l1; ++l)
      for (int b = 0; b < s->d.B; ++b) {
        const int v = ov[(size_t)l * s->d.B + b];
        last_ir[j++] = v < 0 ? -1.f : (float)v / (float)s->d.K;
      }
  }
  return fetch_device_flag(s);
}

int remoe_reuse_mass(remoe_stack* s, int32_t layer, double* mass_sum, uint64_t* pairs, float* last_mass) {
  if (!s || layer < -1 || layer >= s->d.L) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  const size_t n = (size_t)s->d.L * s->d.B;
  std::vector<double> ms(n);
  std::vector<float> lm(n);
  std::vector<unsigned long long> c((size_t)s->d.L * kCounters);
  CK(cudaMemcpy(ms.data(), s->d.mass_sum, n * sizeof(double), cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(lm.data(), s->d.last_mass, n * sizeof(float), cudaMemcpyDeviceToHost));
  CK(cudaMemcpy(c.data(), s->d.counters, c.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  double tot = 0.0;
  uint64_t p = 0;
  size_t j = 0;
  for (int l = 0; l < s->d.L; ++l) {
    if (layer >= 0 && l != layer) continue;
    p += c[(size_t)l * kCounters + 5];
    for (int b = 0; b < s->d.B; ++b) {
      tot += ms[(size_t)l * s->d.B + b];           // fixed order: layer, then sequence
      if (last_mass) last_mass[j++] = lm[(size_t)l * s->d.B + b];
    }
  }
  if (mass_sum) *mass_sum = tot;
  if (pairs) *pairs = p;
  return fetch_device_flag(s);
}

int remoe_expert_load(remoe_stack* s, int32_t layer, uint64_t* counts, double* entropy, double* cv,
                      int32_t* visited) {
  if (!s || layer < -1 || layer >= s->d.L) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  const int N = s->d.N;
  std::vector<unsigned long long> c((size_t)s->d.L * N);
  CK(cudaMemcpy(c.data(), s->d.load, c.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost));
  const int l0 = layer < 0 ? 0 : layer, l1 = layer < 0 ? s->d.L : layer + 1;
  double ent_sum = 0.0, cv_sum = 0.0;
  long seen_sum = 0;
  for (int l = l0; l < l1; ++l) {
    const unsigned long long* n = c.data() + (size_t)l * N;
    if (counts) for (int e = 0; e < N; ++e) counts[(size_t)(l - l0) * N + e] = n[e];
    double tot = 0.0;
    for (int e = 0; e < N; ++e) { tot += (double)n[e]; seen_sum += n[e] ? 1 : 0; }
    if (tot <= 0.0 || N < 2) { ent_sum += 1.0; continue; }        // nothing routed yet: even by convention
    double h = 0.0, var = 0.0;
    const double mean = tot / N;
    for (int e = 0; e < N; ++e) {
      if (n[e]) { const double q = (double)n[e] / tot; h -= q * std::log(q); }
      var += ((double)n[e] - mean) * ((double)n[e] - mean);
    }
    ent_sum += h / std::log((double)N);
    cv_sum += std::sqrt(var / N) / mean;
  }
  const int nl = l1 - l0;
  if (entropy) *entropy = ent_sum / nl;
  if (cv) *cv = cv_sum / nl;
  if (visited) *visited = (int32_t)(seen_sum / nl);
  return fetch_device_flag(s);
}

int remoe_step_history(remoe_stack* s, int32_t first, int32_t count, uint32_t* umiss, uint32_t* tok_hits,
                       int32_t* n_steps) {
  if (!s || first < 0 || count < 0) return REMOE_E_ARG;
  const int32_t have = (int32_t)s->hist_umiss.size();
  if (n_steps) *n_steps = have;
  for (int32_t i = 0; i < count && first + i < have; ++i) {
    if (umiss) umiss[i] = s->hist_umiss[first + i];
    if (tok_hits) tok_hits[i] = s->hist_tok_hits[first + i];
  }
  return REMOE_OK;
}

int remoe_tpot_proxy(const uint32_t* umiss, int32_t n, uint64_t expert_bytes, double bandwidth_gbps, int32_t batch,
                     double tpot_compute_ms, double* io_ms, double* tpot_p50_p95_p99) {
  if (!umiss || n < 1 || batch < 1 || !(bandwidth_gbps > 0.0)) return REMOE_E_ARG;
  std::vector<double> tpot((size_t)n);
  for (int32_t i = 0; i < n; ++i) {
    const double io = (double)umiss[i] * (double)expert_bytes / (bandwidth_gbps * 1e9) * 1000.0;
    if (io_ms) io_ms[i] = io;
    tpot[i] = tpot_compute_ms + io / (double)batch;
  }
  if (tpot_p50_p95_p99) {
    std::sort(tpot.begin(), tpot.end());
    const double q[3] = {0.50, 0.95, 0.99};
    for (int k = 0; k < 3; ++k) {
      const double pos = q[k] * (double)(n - 1);          // linear interpolation between order statistics
      const int32_t lo = (int32_t)pos;
      const int32_t hi = lo + 1 < n ? lo + 1 : lo;
      tpot_p50_p95_p99[k] = tpot[lo] + (pos - (double)lo) * (tpot[hi] - tpot[lo]);
    }
  }
  return REMOE_OK;
}

int remoe_cache_reset(remoe_stack* s) {
  if (!s) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  CK(cudaStreamSynchronize(s->stream));
  CK(cudaStreamSynchronize(s->copy_stream));
  l_host_sync(s, kStCompute);
  l_host_sync(s, kStCopy);
  return reset_state(s);
}

int remoe_set_policy(remoe_stack* s, int32_t policy) {
  if (!s || policy < REMOE_POLICY_LRU || policy > REMOE_POLICY_LFU) return REMOE_E_ARG;
  s->policy = policy;
  return remoe_cache_reset(s);
}

int remoe_set_reroute_beta(remoe_stack* s, float beta) {
  if (!s || !(beta == beta)) return REMOE_E_ARG;
  s->beta = beta;
  return REMOE_OK;
}

int remoe_set_profiling(remoe_stack* s, int32_t on) {
  if (!s) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  int rc = prof_collect(s);
  if (rc != REMOE_OK) return rc;
  s->profiling = on != 0;
  for (int p = 0; p < 2; ++p) {
    s->prof_ms[p] = 0.0;
    s->prof_launches[p] = 0;
    s->prof_bytes[p] = 0;
  }
  return REMOE_OK;
}

int remoe_kernel_time(remoe_stack* s, int32_t phase, double* ms_sum, uint64_t* launches, uint64_t* bytes) {
  if (!s || phase < 0 || phase > 1) return REMOE_E_ARG;
  ON_STACK_DEVICE(s);
  int rc = prof_collect(s);
  if (rc != REMOE_OK) return rc;
  if (ms_sum) *ms_sum = s->prof_ms[phase];
  if (launches) *launches = s->prof_launches[phase];
  if (bytes) *bytes = s->prof_bytes[phase];
  return REMOE_OK;
}

int remoe_order_check_counts(remoe_stack* s, uint64_t* comparisons, uint64_t* violations) {
  if (!s) return REMOE_E_ARG;
  if (comparisons) *comparisons = s->ledger ? s->ledger->checks() : 0;
  if (violations) *violations = s->ledger ? s->ledger->violations() : 0;
  return REMOE_OK;
}

int remoe_launch_count(remoe_stack* s, uint64_t* launches) {
  if (!s || !launches) return REMOE_E_ARG;
  *launches = s->kernel_launches;
  return REMOE_OK;
}

}  // extern "C"

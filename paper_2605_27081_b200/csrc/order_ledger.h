// Host-side ordering check for the step scheduler (plain C++, no CUDA).
//
// The scheduler spreads a decode step over several streams: routing, expert kernels and combine on
// the compute stream (routing of the next step on a route stream in the multi-step call), expert
// fetches on a copy stream, tied together by events.  Two orderings keep the cache slots coherent:
//   - a copy into a slot (or a kernel that rewrites it) must come after every kernel that read the
//     slot's previous contents (write after read), and after the previous write;
//   - a kernel that reads a slot must come after the write that filled it (read after write).
// This ledger replays what the scheduler enqueues -- operations on streams, event records, event
// waits, host waits -- with one vector clock per stream, and checks both orderings for every
// declared access.  It sees only the schedule, never the GPU: a violation means the host code
// enqueued work whose order the streams and events do not guarantee, whether or not the race
// would have shown in that run.  Switched on per stack with REMOE_CHECK_ORDER=1.
#pragma once

#include <array>
#include <cstdint>
#include <string>
#include <unordered_map>
#include <vector>

namespace remoe {

class OrderLedger {
 public:
  static constexpr int kStreams = 4;
  using Clock = std::array<uint64_t, kStreams>;
  struct Op {
    int stream;
    uint64_t index;          // 1-based position on its stream
    Clock seen;              // per stream, the last operation known to precede this one when it was enqueued
  };

  // A new operation (kernel launch or copy) enqueued on `stream`.
  Op op(int stream) {
    Clock& c = clock_[stream];
    for (int s = 0; s < kStreams; ++s) c[s] = c[s] > host_[s] ? c[s] : host_[s];   // enqueued after the host saw those finish
    c[stream] = ++pos_[stream];
    return Op{stream, pos_[stream], c};
  }
  // cudaEventRecord(event, stream): the event stands for everything enqueued on the stream so far
  // and everything that precedes it.
  void record(const void* event, int stream) {
    Clock c = clock_[stream];
    c[stream] = pos_[stream];
    events_[event] = c;
  }
  // cudaStreamWaitEvent(stream, event): later operations of the stream follow what the event stands for.
  void wait(int stream, const void* event) {
    auto it = events_.find(event);
    if (it == events_.end()) return;               // never recorded: the wait is a no-op, as in CUDA
    merge(clock_[stream], it->second);
  }
  // cudaEventSynchronize(event) on the host: whatever is enqueued from now on, on any stream, follows it.
  void host_wait(const void* event) {
    auto it = events_.find(event);
    if (it != events_.end()) merge(host_, it->second);
  }
  // cudaStreamSynchronize(stream) on the host.
  void host_sync(int stream) {
    Clock c = clock_[stream];
    c[stream] = pos_[stream];
    merge(host_, c);
  }

  // `o` reads cell `cell`: the write that filled the cell must precede it.
  bool read(const Op& o, uint64_t cell, const char* what) {
    Cell& c = cells_[cell];
    bool ok = true;
    if (c.written && !before(c.writer, o)) ok = fail("read of cell", cell, what, c.writer, o);
    c.readers.push_back(o);
    return ok;
  }
  // `o` overwrites cell `cell`: every reader of the old contents and the previous write must precede it.
  bool write(const Op& o, uint64_t cell, const char* what) {
    Cell& c = cells_[cell];
    bool ok = true;
    for (const Op& r : c.readers)
      if (!before(r, o)) ok = fail("overwrite of cell", cell, what, r, o);
    if (c.written && !before(c.writer, o)) ok = fail("overwrite of cell", cell, what, c.writer, o);
    c.readers.clear();
    c.writer = o;
    c.written = true;
    return ok;
  }

  uint64_t violations() const { return violations_; }
  const std::string& first_violation() const { return first_; }
  uint64_t checks() const { return checks_; }

 private:
  struct Cell {
    std::vector<Op> readers;     // since the last write
    Op writer{0, 0, {}};
    bool written = false;
  };
  static void merge(Clock& into, const Clock& from) {
    for (int s = 0; s < kStreams; ++s) into[s] = into[s] > from[s] ? into[s] : from[s];
  }
  // does `a` happen before `b` by stream order, event edges or host waits?
  bool before(const Op& a, const Op& b) {
    ++checks_;
    if (a.stream == b.stream) return a.index < b.index;
    return b.seen[a.stream] >= a.index;              // what b's stream had waited for when b was enqueued
  }
  bool fail(const char* kind, uint64_t cell, const char* what, const Op& earlier, const Op& later) {
    if (violations_++ == 0)
      first_ = std::string(kind) + " " + std::to_string(cell) + " (" + what + "): operation " +
               std::to_string(later.index) + " on stream " + std::to_string(later.stream) +
               " is not ordered after operation " + std::to_string(earlier.index) + " on stream " +
               std::to_string(earlier.stream);
    return false;
  }

  Clock clock_[kStreams] = {};
  Clock host_ = {};
  uint64_t pos_[kStreams] = {};
  std::unordered_map<const void*, Clock> events_;
  std::unordered_map<uint64_t, Cell> cells_;
  uint64_t violations_ = 0, checks_ = 0;
  std::string first_;
};

}  // namespace remoe

// Drives the scheduler's ordering ledger with small hand-made schedules (no GPU): a correct two-stream
// fetch schedule passes; the same schedule with one wait left out, a reader enqueued before its fetch, and
// a buffer reused without its release event are each reported.  Prints "ok" and exits 0 on success.
#include <cstdio>
#include <cstdlib>

#include "order_ledger.h"

using remoe::OrderLedger;
enum { kCompute = 0, kCopy = 1, kRoute = 2 };

#define EXPECT(cond)                                                          \
  do {                                                                        \
    if (!(cond)) {                                                            \
      std::printf("FAILED line %d: %s\n", __LINE__, #cond);                   \
      return 1;                                                               \
    }                                                                         \
  } while (0)

// One step of the single-step schedule over slot 7: a kernel of the previous step read it, this step
// routes, fetches a new expert into it on the copy stream and reads it in a miss-phase launch.
static uint64_t one_step(bool wait_for_route, bool wait_for_copy) {
  OrderLedger g;
  int ev_trace, ev_layer;                       // addresses stand in for event handles
  OrderLedger::Op prev = g.op(kCompute);        // previous step's expert kernel
  g.read(prev, 7, "previous step");
  g.op(kCompute);                               // this step's route kernel
  g.record(&ev_trace, kCompute);
  if (wait_for_route) g.wait(kCopy, &ev_trace);
  OrderLedger::Op cp = g.op(kCopy);
  g.write(cp, 7, "fetch");
  g.record(&ev_layer, kCopy);
  if (wait_for_copy) g.wait(kCompute, &ev_layer);
  OrderLedger::Op miss = g.op(kCompute);
  g.read(miss, 7, "miss-phase launch");
  return g.violations();
}

int main() {
  EXPECT(one_step(true, true) == 0);
  EXPECT(one_step(false, true) == 1);           // the copy may overtake the previous step's reader
  EXPECT(one_step(true, false) == 1);           // the kernel may read before the fetch has landed
  EXPECT(one_step(false, false) == 2);

  {  // a host wait orders later work of every stream behind what the event covers
    OrderLedger g;
    int ev;
    OrderLedger::Op k = g.op(kCompute);
    g.read(k, 3, "reader");
    g.record(&ev, kCompute);
    g.host_wait(&ev);
    g.write(g.op(kCopy), 3, "fetch after the host saw the reader finish");
    EXPECT(g.violations() == 0);
    // ... but not behind work enqueued after the event
    OrderLedger::Op k2 = g.op(kCompute);
    g.read(k2, 3, "late reader");               // reads the copy's data without waiting for it
    EXPECT(g.violations() == 1);
    EXPECT(g.first_violation().find("read of cell 3") != std::string::npos);
  }
  {  // transitivity: copy waits for B, B's stream had waited for A
    OrderLedger g;
    int ev_a, ev_b;
    OrderLedger::Op a = g.op(kRoute);
    g.read(a, 1, "A");
    g.record(&ev_a, kRoute);
    g.wait(kCompute, &ev_a);
    g.op(kCompute);
    g.record(&ev_b, kCompute);
    g.wait(kCopy, &ev_b);
    g.write(g.op(kCopy), 1, "fetch");
    EXPECT(g.violations() == 0);
  }
  {  // an event that is recorded again stands for the later record only from then on; a wait taken before does not
    OrderLedger g;
    int ev;
    g.op(kCompute);
    g.record(&ev, kCompute);
    g.wait(kCopy, &ev);
    OrderLedger::Op r = g.op(kCompute);         // enqueued after the record the copy stream waited for
    g.read(r, 9, "reader");
    g.record(&ev, kCompute);
    g.write(g.op(kCopy), 9, "fetch");
    EXPECT(g.violations() == 1);
    g.wait(kCopy, &ev);
    g.write(g.op(kCopy), 9, "fetch");           // same-stream write after write, readers cleared: fine
    EXPECT(g.violations() == 1);
  }
  {  // the multi-step schedule: step t+1's fetch into a slot must wait for step t's resident launch (ev_res) and, if
     // step t fetched into that layer, for its miss-phase launch (ev_miss)
    for (int with_miss_wait = 0; with_miss_wait < 2; ++with_miss_wait) {
      OrderLedger g;
      int ev_route0, ev_res0, ev_copy0, ev_miss0, ev_route1;
      g.op(kRoute); g.record(&ev_route0, kRoute);
      g.wait(kCompute, &ev_route0);
      OrderLedger::Op res0 = g.op(kCompute); g.record(&ev_res0, kCompute);
      g.host_wait(&ev_route0);
      g.op(kRoute); g.record(&ev_route1, kRoute);                     // step 1 routed early
      OrderLedger::Op c0 = g.op(kCopy); g.write(c0, 5, "step 0 fetch");
      g.record(&ev_copy0, kCopy); g.wait(kCompute, &ev_copy0);
      OrderLedger::Op m0 = g.op(kCompute); g.read(m0, 5, "step 0 miss-phase"); g.record(&ev_miss0, kCompute);
      g.read(res0, 4, "step 0 resident");
      // step 1 evicts both slots
      g.wait(kCompute, &ev_route1); g.op(kCompute);
      g.host_wait(&ev_route1);
      g.wait(kCopy, &ev_res0);
      if (with_miss_wait) g.wait(kCopy, &ev_miss0);
      g.write(g.op(kCopy), 4, "step 1 fetch");
      g.write(g.op(kCopy), 5, "step 1 fetch");
      EXPECT(g.violations() == (with_miss_wait ? 0u : 1u));
    }
  }
  std::printf("ok\n");
  return 0;
}

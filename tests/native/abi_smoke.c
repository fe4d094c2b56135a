/* The C ABI used from plain C, no Python and no PyTorch: a tiny float32 stack (1 layer, H = 128, 6 routed
 * experts, top-2, one shared expert, 3 cache slots) is built from a linear congruential generator, stepped
 * through remoe_decode_step_host, and every step's selection, gate weights, output, hit/miss counts and reuse
 * are set against a double-precision restatement written out below (routing: Sec. 3.1; cache: App. A.1-A.2 with
 * LRU; reuse: Eq. 1).  Prints "ok" and exits 0 on success. */
#include <cuda_runtime_api.h>
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include "remoe.h"

enum { L = 1, H = 128, N = 6, K = 2, I = 8, IS = 5, C = 3, STEPS = 12 };

static unsigned long long lcg_state = 12345;
static float lcg_uniform(void) {                       /* (-1, 1) */
  lcg_state = lcg_state * 6364136223846793005ULL + 1442695040888963407ULL;
  return (float)((double)(lcg_state >> 11) / 9007199254740992.0 * 2.0 - 1.0);
}

#define CHECK(cond)                                                   \
  do {                                                                \
    if (!(cond)) {                                                    \
      printf("FAILED line %d: %s\n", __LINE__, #cond);                \
      return 1;                                                       \
    }                                                                 \
  } while (0)

/* y += scale * W_down (silu(W_gate x) * (W_up x)) for one block in the [I, 3, H] layout */
static void expert(const float* blk, int inter, const float* x, double scale, double* y) {
  for (int i = 0; i < inter; ++i) {
    const float *g = blk + (size_t)i * 3 * H, *u = g + H, *d = u + H;
    double zg = 0, zu = 0;
    for (int j = 0; j < H; ++j) { zg += (double)g[j] * x[j]; zu += (double)u[j] * x[j]; }
    const double a = zg / (1.0 + exp(-zg)) * zu * scale;
    for (int j = 0; j < H; ++j) y[j] += a * d[j];
  }
}

int main(void) {
  static float router[N * H], shared[3 * IS * H], x[H], out[H], gw[K];
  static int ids[K];
  float* blocks[N];
  const void* ptrs[N];
  for (int i = 0; i < N * H; ++i) router[i] = lcg_uniform() * 0.3f;
  for (int i = 0; i < 3 * IS * H; ++i) shared[i] = lcg_uniform() * 0.05f;
  for (int e = 0; e < N; ++e) {
    CHECK(cudaMallocHost((void**)&blocks[e], sizeof(float) * 3 * I * H) == cudaSuccess);
    for (int i = 0; i < 3 * I * H; ++i) blocks[e][i] = lcg_uniform() * 0.05f;
    ptrs[e] = blocks[e];
  }

  remoe_shape sh;
  memset(&sh, 0, sizeof sh);
  sh.n_layers = L; sh.hidden = H; sh.n_routed = N; sh.top_k = K; sh.inter_routed = I;
  sh.n_shared = 1; sh.inter_shared = IS; sh.weight_dtype = REMOE_F32; sh.batch = 1;
  remoe_stack* st = NULL;
  CHECK(remoe_stack_create(&sh, K - 1, NULL, &st) == REMOE_E_CAPACITY && st == NULL);
  CHECK(remoe_stack_create(&sh, C, NULL, &st) == REMOE_OK && st != NULL);
  CHECK(remoe_decode_step_host(st, x, out, ids, gw) == REMOE_E_NOT_LOADED);        /* nothing loaded yet */
  CHECK(remoe_load_router(st, 0, router, NULL) == REMOE_OK);
  CHECK(remoe_load_shared(st, 0, 0, shared) == REMOE_OK);
  CHECK(remoe_load_experts_host(st, 0, 0, N, ptrs) == REMOE_OK);
  {
    const void* pageable = router;                      /* ordinary host memory is refused */
    CHECK(remoe_load_experts_host(st, 0, 0, 1, &pageable) == REMOE_E_NOT_PINNED);
    CHECK(remoe_load_experts_host(st, 0, 0, 1, ptrs) == REMOE_OK);
  }

  /* the cache, restated: resident set with last-touch stamps */
  int resident[C], n_res = 0;
  long stamp[C], clock = 0;
  int prev[K], have_prev = 0;
  uint64_t hits = 0, misses = 0, overlap = 0, pairs = 0;

  for (int t = 0; t < STEPS; ++t) {
    for (int j = 0; j < H; ++j) x[j] = (t % 3 == 2) ? x[j] : lcg_uniform();   /* every third step repeats its input */
    CHECK(remoe_decode_step_host(st, x, out, ids, gw) == REMOE_OK);

    /* routing: logits, softmax, the K largest by (logit descending, index ascending) */
    double z[N], p[N], zmax = -1e300, sum = 0;
    for (int e = 0; e < N; ++e) {
      z[e] = 0;
      for (int j = 0; j < H; ++j) z[e] += (double)router[e * H + j] * x[j];
      if (z[e] > zmax) zmax = z[e];
    }
    for (int e = 0; e < N; ++e) { p[e] = exp(z[e] - zmax); sum += p[e]; }
    int want[K], taken[N] = {0};
    for (int k = 0; k < K; ++k) {
      int best = -1;
      for (int e = 0; e < N; ++e)
        if (!taken[e] && (best < 0 || z[e] > z[best])) best = e;
      taken[best] = 1;
      want[k] = best;
    }
    for (int k = 0; k < K; ++k) {
      CHECK(ids[k] == want[k]);
      CHECK(fabs(gw[k] - p[want[k]] / sum) <= 1e-6);
    }
    /* output: gate-weighted routed experts plus the shared expert */
    double y[H];
    for (int j = 0; j < H; ++j) y[j] = 0;
    for (int k = 0; k < K; ++k) expert(blocks[want[k]], I, x, p[want[k]] / sum, y);
    expert(shared, IS, x, 1.0, y);
    double ymax = 0, emax = 0;
    for (int j = 0; j < H; ++j) {
      if (fabs(y[j]) > ymax) ymax = fabs(y[j]);
      if (fabs(out[j] - y[j]) > emax) emax = fabs(out[j] - y[j]);
    }
    CHECK(emax <= 1e-4 * ymax);
    /* cache: classify against the state before the step, touch hits in order, then admit misses (LRU) */
    int hit[K], slot_of[K];
    for (int k = 0; k < K; ++k) {
      hit[k] = 0;
      for (int s = 0; s < n_res; ++s)
        if (resident[s] == want[k]) { hit[k] = 1; slot_of[k] = s; }
    }
    for (int k = 0; k < K; ++k)
      if (hit[k]) { stamp[slot_of[k]] = ++clock; ++hits; }
    for (int k = 0; k < K; ++k) {
      if (hit[k]) continue;
      ++misses;
      int s;
      if (n_res < C) {
        s = n_res++;
      } else {
        s = -1;
        for (int c = 0; c < C; ++c) {
          int used_now = 0;
          for (int q = 0; q < K; ++q) used_now |= resident[c] == want[q];
          if (!used_now && (s < 0 || stamp[c] < stamp[s])) s = c;
        }
      }
      resident[s] = want[k];
      stamp[s] = ++clock;
    }
    if (have_prev) {
      for (int a = 0; a < K; ++a)
        for (int b = 0; b < K; ++b) overlap += want[a] == prev[b];
      ++pairs;
    }
    memcpy(prev, want, sizeof prev);
    have_prev = 1;
  }

  remoe_cache_counters cc;
  CHECK(remoe_cache_stats(st, -1, &cc) == REMOE_OK);
  CHECK(cc.uniq_hits == hits && cc.uniq_misses == misses && cc.tok_hits == hits && cc.tok_misses == misses);
  CHECK(hits + misses == (uint64_t)L * K * STEPS && cc.steps == STEPS);
  CHECK(cc.h2d_bytes == misses * sizeof(float) * 3 * I * H);
  uint64_t ov = 0, pr = 0;
  CHECK(remoe_reuse_stats(st, -1, &ov, &pr, NULL) == REMOE_OK);
  CHECK(ov == overlap && pr == pairs && pr == STEPS - 1);
  CHECK(hits > 0 && misses > (uint64_t)K);        /* both kinds occurred */
  CHECK(strcmp(remoe_strerror(REMOE_E_CAPACITY), "cache capacity below top_k") == 0);
  remoe_stack_destroy(st);
  for (int e = 0; e < N; ++e) cudaFreeHost(blocks[e]);
  printf("ok\n");
  return 0;
}

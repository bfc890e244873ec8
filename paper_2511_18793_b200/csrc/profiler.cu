// Launch counting and optional per-kernel-class CUDA-event timing.  Process-wide, not thread-safe: meant for
// one benchmarking thread.
#include <stdlib.h>

#include <vector>

#include "common.cuh"

namespace nz {

namespace {
struct Pair { cudaEvent_t a, b; int cls; };
unsigned long long g_total = 0;
bool g_on = false;
long long g_launches[kcCount] = {0};
std::vector<Pair> g_pairs;
size_t g_used = 0;
}  // namespace

LaunchScope::LaunchScope(int cls_, cudaStream_t st_, int n_launches) : cls(cls_), st(st_), slot(-1) {
  g_total += (unsigned long long)n_launches;
  g_launches[cls] += n_launches;
  if (!g_on) return;
  if (g_used == g_pairs.size()) {
    Pair p{};
    if (cudaEventCreate(&p.a) != cudaSuccess || cudaEventCreate(&p.b) != cudaSuccess) return;
    g_pairs.push_back(p);
  }
  slot = (int)g_used++;
  g_pairs[slot].cls = cls;
  cudaEventRecord(g_pairs[slot].a, st);
}

LaunchScope::~LaunchScope() {
  if (slot >= 0) cudaEventRecord(g_pairs[slot].b, st);
}

bool pdl_enabled() {
  static const bool on = getenv("NEZHA_NO_PDL") == nullptr;
  return on;
}

unsigned long long profile_total_launches() { return g_total; }

bool profile_is_on() { return g_on; }

// Launch counts per class so far (for code that replays a captured CUDA graph: it snapshots before and after the
// capture and adds the difference on every replay).
void profile_counts(long long* out) {
  for (int i = 0; i < kcCount; ++i) out[i] = g_launches[i];
}
void profile_add(const long long* delta) {
  for (int i = 0; i < kcCount; ++i) { g_launches[i] += delta[i]; g_total += (unsigned long long)delta[i]; }
}

void profile_enable(bool on) {
  g_on = on;
  g_used = 0;
}

// The caller has synchronised the stream(s) the scopes ran on.
void profile_read(nezha_profile* out) {
  for (int i = 0; i < NEZHA_PROFILE_CLASSES; ++i) { out->launches[i] = 0; out->ms[i] = 0.0; }
  for (int i = 0; i < kcCount; ++i) { out->launches[i] = g_launches[i]; g_launches[i] = 0; }
  for (size_t i = 0; i < g_used; ++i) {
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, g_pairs[i].a, g_pairs[i].b) == cudaSuccess) out->ms[g_pairs[i].cls] += ms;
  }
  g_used = 0;
}

}  // namespace nz

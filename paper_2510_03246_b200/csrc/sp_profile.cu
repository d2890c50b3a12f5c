// Launch counter and optional CUDA-event timing of the library's kernels, per kernel kind.
#include <atomic>
#include <vector>

#include "sp_common.cuh"

namespace sp {
namespace {

constexpr int kMaxSlots = 65536;
struct Slot {
  cudaEvent_t start, stop;
  int kind;
  double flops, bytes;
};
std::atomic<long long> g_launches{0};
std::atomic<int> g_reproducible{0};
std::atomic<long long> g_wait_budget{0};
int g_enabled = 0;   // 0 off, 1 outermost scopes only, 2 every scope (nested ones are then counted twice)
std::vector<Slot> g_slots;
int g_used = 0;
thread_local int g_depth = 0;
thread_local const int32_t* g_skip = nullptr;

}  // namespace

long long wait_budget_cycles() { return g_wait_budget.load(std::memory_order_relaxed); }

bool reproducible_mode() { return g_reproducible.load(std::memory_order_relaxed) != 0; }

const int32_t* skip_flag() { return g_skip; }
SkipScope::SkipScope(const int32_t* flag) { g_skip = flag; }
SkipScope::~SkipScope() { g_skip = nullptr; }

void count_launch(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

ProfScope::ProfScope(int kind, double flops, double bytes, cudaStream_t s) : slot(-1), stream(s) {
  const bool nested = g_depth++ > 0;
  if (!g_enabled || (nested && g_enabled < 2) || g_used >= kMaxSlots) return;
  if ((int)g_slots.size() <= g_used) {
    Slot sl;
    if (cudaEventCreate(&sl.start) != cudaSuccess || cudaEventCreate(&sl.stop) != cudaSuccess) return;
    g_slots.push_back(sl);
  }
  slot = g_used++;
  g_slots[slot].kind = kind;
  g_slots[slot].flops = flops;
  g_slots[slot].bytes = bytes;
  cudaEventRecord(g_slots[slot].start, stream);
}

ProfScope::~ProfScope() {
  --g_depth;
  if (slot >= 0) cudaEventRecord(g_slots[slot].stop, stream);
}

}  // namespace sp

extern "C" {

sp_status sp_set_reproducible(int32_t on) {
  sp::g_reproducible.store(on ? 1 : 0);
  return SP_OK;
}
sp_status sp_set_wait_budget(int64_t cycles) {
  if (cycles < 0) return SP_ERR_INVALID_ARG;
  sp::g_wait_budget.store((long long)cycles);
  return SP_OK;
}

int32_t sp_get_reproducible(void) { return sp::g_reproducible.load(); }

int64_t sp_launch_count(void) { return (int64_t)sp::g_launches.load(); }

sp_status sp_profile_begin(int32_t enable) {
  sp::g_enabled = enable;
  sp::g_used = 0;
  sp::g_launches.store(0);
  return SP_OK;
}

int32_t sp_profile_kinds(void) { return sp::PK_COUNT; }

const char* sp_profile_kind_name(int32_t kind) {
  static const char* names[sp::PK_COUNT] = {"gemm_tc", "gemm_simt", "solve_phase", "fused_update", "prep_h",
                                            "scores", "topk_select", "elementwise", "allocate", "chol_diag",
                                            "panel_apply", "gemm_tc_shared", "conditional"};
  return (kind >= 0 && kind < sp::PK_COUNT) ? names[kind] : "unknown";
}

sp_status sp_profile_read(double* out_host) {
  if (!out_host) return SP_ERR_INVALID_ARG;
  for (int i = 0; i < sp::PK_COUNT * 4; ++i) out_host[i] = 0.0;
  for (int i = 0; i < sp::g_used; ++i) {
    const sp::Slot& s = sp::g_slots[i];
    float ms = 0.f;
    if (cudaEventElapsedTime(&ms, s.start, s.stop) != cudaSuccess) return SP_ERR_CUDA;
    double* o = out_host + s.kind * 4;
    o[0] += 1.0;
    o[1] += (double)ms;
    o[2] += s.flops;
    o[3] += s.bytes;
  }
  return SP_OK;
}

}  // extern "C"

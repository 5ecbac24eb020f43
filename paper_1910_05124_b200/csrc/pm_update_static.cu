// pm_update_flat_static: the stand-alone fused update for callers that cannot allocate device memory.
//
// Some hosts of this library run where cudaMalloc is off limits: inside a framework whose caching
// allocator owns the whole device, in a real-time loop that forbids allocation after start-up, or in a
// plug-in that is handed tensors but no allocator.  pm_update_flat asks such a caller for a device
// workspace it has no way to provide.  This variant keeps that workspace (the per-stage table the
// scheduler and the update kernel read) in a fixed array that is part of the library image, so the call
// needs only the arenas themselves.
#include <mutex>
#include <string>
#include <cstring>

#include "pm_update.cuh"

using namespace pm;

#define PM_STATIC_MAX_STAGES 256

namespace {

inline uint64_t align_up(uint64_t v, uint64_t a) { return (v + a - 1) / a * a; }

constexpr uint64_t table_bytes(uint64_t P) {
  uint64_t w = 0;
  w = (w + sizeof(StageSched) * P + 255) / 256 * 256;
  w = (w + sizeof(StageDyn) * P + 255) / 256 * 256;
  w = (w + sizeof(int64_t) * P + 255) / 256 * 256;
  w = (w + sizeof(uint32_t) * P + 255) / 256 * 256;
  w = (w + sizeof(uint32_t) * P + 255) / 256 * 256;
  return w;
}
constexpr uint64_t kScratchBytes = table_bytes(PM_STATIC_MAX_STAGES);

// The scratch itself.  Every GPU that loads the library holds these bytes until the process exits.
// In host code this name is only a handle for the runtime; the address a kernel can use comes from
// cudaGetSymbolAddress, looked up once per device below.
static __device__ __align__(256) unsigned char g_static_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};
thread_local std::string g_static_error;

// host staging for the table; fixed size so that the call performs no allocation of any kind
thread_local unsigned char g_host_table[kScratchBytes];

}  // namespace

extern "C" {

const char* pm_update_flat_static_last_error(void) { return g_static_error.c_str(); }

int32_t pm_update_flat_static_max_stages(void) { return PM_STATIC_MAX_STAGES; }

pm_status pm_update_flat_static(const pm_arenas* arenas, const uint64_t* stage_offsets, const uint64_t* stage_counts,
                                const int32_t* tau_fwd, const int32_t* tau_bkwd, int32_t n_stages,
                                const pm_config* cfg, int64_t k, void* stream) {
  auto fail = [](pm_status s, const char* msg) { g_static_error = msg; return s; };
  if (!arenas || !stage_offsets || !stage_counts || !tau_fwd || !tau_bkwd || !cfg) return fail(PM_ERR_INVALID_ARG, "null argument");
  if (n_stages < 1) return fail(PM_ERR_INVALID_ARG, "n_stages must be positive");
  if (n_stages > PM_STATIC_MAX_STAGES)
    return fail(PM_ERR_NOMEM, "pm_update_flat_static holds its stage table in a fixed device array sized for at most "
                              "256 stages; use pm_update_flat with a caller-provided workspace for more");
  if (k < 0) return fail(PM_ERR_INVALID_ARG, "k must be >= 0");
  if (cfg->optimizer != PM_SGDM && cfg->optimizer != PM_ADAM) return fail(PM_ERR_INVALID_ARG, "unknown optimizer");
  if (!arenas->w || !arenas->m || !arenas->delta || !arenas->grad || (cfg->optimizer == PM_ADAM && !arenas->s))
    return fail(PM_ERR_INVALID_ARG, "missing arena");
  if (cfg->alpha_by_step && cfg->alpha_len < 1) return fail(PM_ERR_INVALID_ARG, "alpha_len must be >= 1 with alpha_by_step");

  // once per device, with that device current: ask the runtime where the array lives on this GPU
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(PM_ERR_CUDA, cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(PM_ERR_UNSUPPORTED, "device ordinal beyond the table of static scratch addresses");
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_scratch_ptr[dev] == nullptr) {
      void* p = nullptr;
      e = cudaGetSymbolAddress(&p, g_static_scratch);
      if (e != cudaSuccess || p == nullptr) return fail(PM_ERR_CUDA, e != cudaSuccess ? cudaGetErrorString(e) : "null symbol address");
      g_scratch_ptr[dev] = p;
    }
    scratch = g_scratch_ptr[dev];
  }

  const uint64_t P = (uint64_t)n_stages;
  const uint64_t need = table_bytes(P);
  const uint64_t off_sched = 0, off_dyn = align_up(sizeof(StageSched) * P, 256);
  const uint64_t off_nupd = align_up(off_dyn + sizeof(StageDyn) * P, 256);
  const uint64_t off_b = align_up(off_nupd + sizeof(int64_t) * P, 256);
  const uint64_t off_e = align_up(off_b + sizeof(uint32_t) * P, 256);
  // the array keeps whatever the previous call left: rebuild the whole table, zero counters included
  std::memset(g_host_table, 0, need);
  StageSched* sc = (StageSched*)(g_host_table + off_sched);
  uint32_t* b64 = (uint32_t*)(g_host_table + off_b);
  uint32_t* e64 = (uint32_t*)(g_host_table + off_e);
  uint64_t prev_end = 0;
  for (int i = 0; i < n_stages; ++i) {
    if (stage_offsets[i] % PM_ALIGN_ELEMS) return fail(PM_ERR_INVALID_ARG, "stage offsets must be multiples of 64 elements");
    if (stage_offsets[i] < prev_end) return fail(PM_ERR_INVALID_ARG, "stage slices must ascend without overlap");
    if (tau_fwd[i] < 0 || tau_bkwd[i] < 0 || tau_bkwd[i] > tau_fwd[i]) return fail(PM_ERR_INVALID_ARG, "need 0 <= tau_bkwd <= tau_fwd");
    if (stage_counts[i] > arenas->count || stage_offsets[i] > arenas->count - stage_counts[i])      // also catches a sum that would wrap
      return fail(PM_ERR_NOMEM, "stage slice exceeds the arenas");
    uint64_t end = align_up(stage_offsets[i] + stage_counts[i], PM_ALIGN_ELEMS);
    if (end > arenas->count) return fail(PM_ERR_NOMEM, "stage slice exceeds the arenas");
    prev_end = end;
    sc[i] = StageSched{tau_fwd[i], tau_fwd[i] - tau_bkwd[i], 1, 1, 0, 0};
    b64[i] = (uint32_t)(stage_offsets[i] / 64);
    e64[i] = (uint32_t)(end / 64);
  }
  cudaStream_t st = (cudaStream_t)stream;
  char* ws = (char*)scratch;
  e = cudaMemcpyAsync(ws, g_host_table, need, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return fail(PM_ERR_CUDA, cudaGetErrorString(e));
  HyperDev hp{};
  hp.optimizer = cfg->optimizer; hp.t1 = cfg->t1_enable; hp.t2 = cfg->t2_enable; hp.n_stages = n_stages;
  hp.K = cfg->t1_K > 0 ? cfg->t1_K : 1; hp.D = cfg->t2_D;
  hp.alpha_const = cfg->alpha_by_step ? cfg->alpha_by_step[k < cfg->alpha_len ? k : cfg->alpha_len - 1] : cfg->alpha_const;
  hp.alpha_tab = nullptr; hp.alpha_len = 0;
  hp.beta1 = cfg->beta1; hp.beta2 = cfg->beta2; hp.eps = cfg->eps;
  e = launch_schedule((const StageSched*)(ws + off_sched), (const int64_t*)(ws + off_nupd), (StageDyn*)(ws + off_dyn), hp, 0, 0, k, st);
  if (e != cudaSuccess) return fail(PM_ERR_CUDA, cudaGetErrorString(e));
  ArenasDev a{arenas->w, arenas->m, arenas->s, arenas->delta, arenas->grad, (__nv_bfloat16*)arenas->w_lp, arenas->count};
  e = launch_update(a, (const uint32_t*)(ws + off_b), (const uint32_t*)(ws + off_e), (const StageDyn*)(ws + off_dyn),
                    (int64_t*)(ws + off_nupd), n_stages, e64[n_stages - 1], cfg->optimizer, cfg->beta1, cfg->beta2, cfg->eps, st);
  if (e != cudaSuccess) return fail(PM_ERR_CUDA, cudaGetErrorString(e));
  return PM_OK;
}

}  // extern "C"

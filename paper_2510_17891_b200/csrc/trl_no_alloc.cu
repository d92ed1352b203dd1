// trl_pg_loss_fwd_static: the clipped-surrogate call for callers that cannot hand over a
// workspace because they cannot allocate one.
//
// Who that is: an RL trainer that gave the whole device to its own memory arena at start-up
// (a later cudaMalloc fails or fragments the arena), and a step loop that must not stall
// (cudaMalloc and cudaFree synchronise the whole device).  Such a caller still owns its
// inputs and outputs, but has nowhere to get the few KB of partial sums that
// trl_pg_loss_fwd keeps between its two kernels.  Here those live in a fixed array inside
// the library image instead.
#include <mutex>

#include "trl_internal.h"

namespace {

// One slot = the four partial sums of one (rollout, token tile) pair.  1 MiB per GPU that
// loads the library, held until the process exits.
constexpr int kStaticLossSlots = 65536;
static __device__ __align__(256) float g_loss_partials[kStaticLossSlots * 4];

constexpr int kMaxDevices = 64;
float* g_partials_addr[kMaxDevices] = {};
std::mutex g_setup_mutex;

// The array's name is only a handle in host code; kernels need its device address, which
// differs per device.  Looked up once per device, with that device current.
int partials_for_current_device(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return TRL_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_partials_addr[dev]) {
    float* p = nullptr;
    if (cudaGetSymbolAddress((void**)&p, g_loss_partials) != cudaSuccess || !p) return TRL_ERR_CUDA;
    g_partials_addr[dev] = p;
  }
  *out = g_partials_addr[dev];
  return TRL_OK;
}

}  // namespace

extern "C" int trl_pg_loss_fwd_static(const float* logp, const float* old_logp, const float* adv, const uint8_t* seg,
                                      const int32_t* len, int P, int G, int T, trl_pg_config cfg, float* loss,
                                      float* g, float* stats, int32_t* status_dev, void* stream) {
  (void)status_dev;
  if (!logp || !old_logp || !adv || !seg || !len || !loss || !g) return TRL_ERR_INVALID_ARG;
  if (P <= 0 || G <= 0 || T <= 0 || (long)P * G > 65535 || (long)P * G * T >= (1L << 31)) return TRL_ERR_SHAPE;
  if (!(cfg.eps_lo >= 0.f) || !(cfg.eps_hi >= 0.f) || !(cfg.alpha >= 0.f) || (cfg.clip_form & ~1) || (cfg.agg_mode & ~1))
    return TRL_ERR_INVALID_ARG;
  if ((((uintptr_t)logp | (uintptr_t)old_logp | (uintptr_t)adv | (uintptr_t)seg | (uintptr_t)g) & 15) != 0 ||
      (((uintptr_t)len | (uintptr_t)loss | (uintptr_t)stats) & 3) != 0)
    return TRL_ERR_INVALID_ARG;          // same alignment contract as trl_pg_loss_fwd
  // size limit of the built-in scratch: P*G*ceil(T/16384) slots
  if ((long)P * G * trl::pg_loss_tiles(T) > kStaticLossSlots) return TRL_ERR_WORKSPACE_TOO_SMALL;
  int major = 0, dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return TRL_ERR_CUDA;
  if (major != 10) return TRL_ERR_ARCH;
  float* partials = nullptr;
  if (int e = partials_for_current_device(&partials)) return e;
  // Every slot the second kernel reads is written by the first one in this same call, so
  // nothing left over from an earlier call is ever read and nothing needs clearing.
  trl::launch_pg_loss(logp, old_logp, adv, seg, len, P, G, T, cfg, loss, g, stats, partials, nullptr, 0,
                      (cudaStream_t)stream);
  return cudaGetLastError() == cudaSuccess ? TRL_OK : TRL_ERR_CUDA;
}

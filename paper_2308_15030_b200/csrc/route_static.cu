// Routing-only entry point that allocates nothing: its scratch lives in a file-scope
// device array instead of a cudaMalloc'ed workspace.  See swapmoe_route_static in
// include/swapmoe.h for who needs this and for the limits.
#include "../../include/swapmoe.h"

#include <cuda_runtime.h>

#include <mutex>

#include "common.cuh"
#include "permute.cuh"
#include "router_gate.cuh"

using namespace swapmoe;

namespace {

constexpr int kStaticMaxTokens = SWAPMOE_ROUTE_STATIC_MAX_TOKENS;
constexpr int kStaticMaxCta = (kStaticMaxTokens + kTokTile - 1) / kTokTile;
constexpr int kStaticMaxPairs = kStaticMaxTokens * kMaxTopK;
constexpr int kStaticTileRows = 64;   // row-tile height used for the (unused) tile list
constexpr int kStaticMaxTiles = kStaticMaxPairs / kStaticTileRows + kMaxSlots;

// Layout of the scratch array (all offsets multiples of 256 bytes).
constexpr size_t kOffTicket = 0;                                          // unsigned [1]
constexpr size_t kOffPhys = 256;                                          // int32 [kMaxSlots]
constexpr size_t kOffNTiles = kOffPhys + 256;                             // int32 [1]
constexpr size_t kOffPad = kOffNTiles + 256;                              // int32 [kMaxSlots + 1]
constexpr size_t kOffHist = kOffPad + 512;                                // int32 [cta][K]
constexpr size_t kOffImp = kOffHist + sizeof(int32_t) * kStaticMaxCta * kMaxSlots;   // float [cta][E]
constexpr size_t kOffTiles = kOffImp + sizeof(float) * kStaticMaxCta * kMaxE;        // TileDesc [tiles]
constexpr size_t kScratchBytes = kOffTiles + ((sizeof(TileDesc) * kStaticMaxTiles + 255) / 256) * 256;

// Every GPU that loads this library holds this array (about 0.35 MB) until the process exits.
static __device__ __align__(256) unsigned char g_route_scratch[kScratchBytes];

// In host code `g_route_scratch` is only a host-side stand-in for the symbol, not a
// device address; the real address is looked up once per device and cached here.
constexpr int kMaxDevices = 64;
unsigned char* g_scratch_dev[kMaxDevices] = {nullptr};
std::mutex g_scratch_mutex;

int32_t scratch_for_current_device(unsigned char** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) { cudaGetLastError(); return SWAPMOE_ERR_CUDA; }
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_dev[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_route_scratch) != cudaSuccess || !p) { cudaGetLastError(); return SWAPMOE_ERR_CUDA; }
    // large expert counts need more dynamic shared memory than the default limit
    if (router_gate_set_smem_limit<float>() != cudaSuccess || router_gate_set_smem_limit<bf16>() != cudaSuccess) {
      cudaGetLastError();
      return SWAPMOE_ERR_CUDA;
    }
    g_scratch_dev[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_dev[dev];
  return SWAPMOE_OK;
}

}  // namespace

extern "C" int32_t swapmoe_route_static(const void* x_dev, const void* Wr_dev, const int32_t* expert_to_slot_dev,
                                        const float* enorm_dev, int32_t n_tokens, int32_t d_model, int32_t E,
                                        int32_t top_k, int32_t K, int32_t dtype, int32_t renorm_topk,
                                        float* logits_dev, int32_t* uidx_dev, float* ugate_dev, int32_t* midx_dev,
                                        float* mgate_dev, int32_t* slot_dev, float* xnorm_dev, int32_t* count_dev,
                                        int32_t* offset_dev, float* imp_dev, void* stream) {
  if (n_tokens < 0 || d_model < 1 || E < 1 || top_k < 1 || K < top_k || K > E) return SWAPMOE_ERR_INVALID_ARG;
  if (dtype != SWAPMOE_F32 && dtype != SWAPMOE_BF16) return SWAPMOE_ERR_INVALID_ARG;
  if (renorm_topk != 0 && renorm_topk != 1) return SWAPMOE_ERR_INVALID_ARG;
  if (n_tokens > kStaticMaxTokens) return SWAPMOE_ERR_TOO_MANY_TOKENS;   // beyond what the fixed scratch holds
  if (E > kMaxE || K > kMaxSlots || top_k > kMaxTopK || d_model % 64) return SWAPMOE_ERR_UNSUPPORTED;
  if (n_tokens == 0) return SWAPMOE_OK;
  if (!x_dev || !Wr_dev || !expert_to_slot_dev || !enorm_dev || !logits_dev || !uidx_dev || !ugate_dev ||
      !midx_dev || !mgate_dev || !slot_dev || !xnorm_dev || !count_dev || !offset_dev || !imp_dev)
    return SWAPMOE_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(x_dev) | reinterpret_cast<uintptr_t>(Wr_dev)) & 15) return SWAPMOE_ERR_INVALID_ARG;

  unsigned char* s = nullptr;
  const int32_t rc = scratch_for_current_device(&s);
  if (rc != SWAPMOE_OK) return rc;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The array keeps whatever the previous call left: the ticket counter and the slot->arena
  // table (unused here, all zero) must start at zero, everything else is overwritten.
  if (cudaMemsetAsync(s + kOffTicket, 0, kOffNTiles + 256, st) != cudaSuccess) { cudaGetLastError(); return SWAPMOE_ERR_CUDA; }

  const int n_cta = (n_tokens + kTokTile - 1) / kTokTile;
  RouterArgs ra;
  ra.x = x_dev; ra.Wr = Wr_dev; ra.ext_logits = nullptr; ra.e2s = expert_to_slot_dev; ra.enorm = enorm_dev;
  ra.logits = logits_dev; ra.uidx = uidx_dev; ra.ugate = ugate_dev; ra.midx = midx_dev; ra.mgate = mgate_dev;
  ra.slot = slot_dev; ra.xnorm = xnorm_dev;
  ra.cta_hist = reinterpret_cast<int32_t*>(s + kOffHist);
  ra.cta_imp = reinterpret_cast<float*>(s + kOffImp);
  ra.cta_cnt = nullptr; ra.cta_mimp = nullptr;
  ra.T = n_tokens; ra.d = d_model; ra.E = E; ra.k = top_k; ra.K = K; ra.renorm = renorm_topk;
  ScanArgs& sa = ra.scan;
  sa.cta_hist = ra.cta_hist; sa.cta_imp = ra.cta_imp;
  sa.phys_slot = reinterpret_cast<const int32_t*>(s + kOffPhys);
  sa.cta_base = nullptr;                       // per-CTA running counts: only a permutation would need them
  sa.count = count_dev; sa.offset = offset_dev;
  sa.pad_offset = reinterpret_cast<int32_t*>(s + kOffPad);
  sa.tiles = reinterpret_cast<TileDesc*>(s + kOffTiles);
  sa.n_tiles = reinterpret_cast<int32_t*>(s + kOffNTiles);
  sa.imp = imp_dev;
  sa.ticket = reinterpret_cast<unsigned*>(s + kOffTicket);
  sa.tiles_b = nullptr; sa.n_tiles_b = nullptr; sa.tile_rows_b = 0; sa.touched = nullptr;
  sa.cta_cnt = nullptr; sa.cta_mimp = nullptr; sa.s2e = nullptr; sa.cnt = nullptr; sa.mimp = nullptr;
  sa.n_cta = n_cta; sa.K = K; sa.E = E; sa.tile_rows = kStaticTileRows;
  if (dtype == SWAPMOE_BF16)
    router_gate_fn<bf16>(E)<<<n_cta, 256, router_smem_bytes(E), st>>>(ra);
  else
    router_gate_fn<float>(E)<<<n_cta, 256, router_smem_bytes(E), st>>>(ra);
  return cudaGetLastError() == cudaSuccess ? SWAPMOE_OK : SWAPMOE_ERR_CUDA;
}

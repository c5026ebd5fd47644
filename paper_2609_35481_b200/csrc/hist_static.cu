// Histogram entry point for callers that cannot allocate device memory.
//
// Some hosts of this library own no allocator they may call on the planning path: a plugin that
// runs inside another framework's stream callback or capture region, a process whose memory pool
// was sized and frozen at start-up, a harness that forbids cudaMalloc after initialisation.  They
// cannot hand over the workspace topoep_histogram needs for its per-tile counts.  This variant
// keeps that scratch in a fixed array inside the library image instead.
//
// The array lives in every CUDA context that loads the library, for the life of the context.
// Host code must not pass the symbol itself to a kernel (on the host the name is only a
// stand-in for the device object); the device address is taken once per device with
// cudaGetSymbolAddress and cached.
#include <algorithm>
#include <mutex>

#include "topoep_internal.cuh"

namespace {

constexpr size_t kScratchBytes = 8u << 20;   // 8 MiB: flags word + per-tile counts
constexpr size_t kFlagsBytes = 256;          // first 256 bytes: status word, rest unused
constexpr int kStaticTileIds = 4096;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_hist_scratch[kScratchBytes];

std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices];   // device address of g_hist_scratch, per device ordinal
int g_sms[kMaxDevices];              // SM count of the device (launch shapes)

// Device address of the scratch array on the current device; resolved on the first call there.
// The cache is keyed by the device ordinal, i.e. it assumes the runtime's primary context: a
// program that drives the same device through a second, driver-API context would be handed the
// primary context's address there.
cudaError_t scratch_address(void** out, int* sms) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_scratch_addr[dev]) {
    void* ptr = nullptr;
    e = cudaGetSymbolAddress(&ptr, g_hist_scratch);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&g_sms[dev], cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = ptr;
  }
  *out = g_scratch_addr[dev];
  *sms = g_sms[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" int topoep_histogram_static(const int32_t* dev_topk_ids, int batch, int ranks,
                                        int tokens_per_rank, int top_k, int experts,
                                        int32_t* dev_omega, uint32_t* dev_flags,
                                        topoep_stream_t stream) {
  using namespace topoep;
  if (batch < 0 || ranks < 1 || tokens_per_rank < 0 || top_k < 1 || experts < 1)
    return TOPOEP_ERR_CONFIG;
  if (batch == 0) return TOPOEP_OK;
  if (!dev_omega || (!dev_topk_ids && tokens_per_rank > 0)) return TOPOEP_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(dev_topk_ids) & 3u) || (reinterpret_cast<uintptr_t>(dev_omega) & 3u) ||
      (reinterpret_cast<uintptr_t>(dev_flags) & 3u))
    return TOPOEP_ERR_ALIGN;
  if (batch > 65535 || ranks > 65535 || ((size_t)experts + 1) * sizeof(int) > 48 * 1024)
    return TOPOEP_ERR_CONFIG;
  const long long n_ids = (long long)tokens_per_rank * top_k;
  if (n_ids >= (1ll << 31)) return TOPOEP_ERR_CONFIG;
  const long long tiles = std::max(1ll, (n_ids + kStaticTileIds - 1) / kStaticTileIds);
  // 4 * batch * ranks * tiles * experts bytes of tile counts must fit behind the flag word.
  // Checked by division, one factor at a time: the product itself can exceed 64 bits for sizes
  // the range checks above let through.
  {
    unsigned long long cells = (kScratchBytes - kFlagsBytes) / 4;   // 32-bit counts that fit
    cells /= (unsigned long long)experts;
    cells /= (unsigned long long)tiles;
    cells /= (unsigned long long)ranks;
    if ((unsigned long long)batch > cells) return TOPOEP_ERR_SCRATCH;   // no fallback
  }

  void* base = nullptr;
  int sms = 0;
  cudaError_t e = scratch_address(&base, &sms);
  if (e != cudaSuccess) return TOPOEP_ERR_CUDA;
  uint32_t* flags = dev_flags ? dev_flags : static_cast<uint32_t*>(base);
  // the status word only ever gets bits OR-ed in, so it must start at zero for this call; the
  // tile counts need no clearing: every cell this call reads it has written first
  e = cudaMemsetAsync(flags, 0, sizeof(uint32_t), stream);
  if (e != cudaSuccess) return TOPOEP_ERR_CUDA;

  HistParams hp = {};
  hp.d.R = ranks;
  hp.d.E = experts;
  hp.d.k = top_k;
  hp.d.sms = sms;
  hp.rank_first = 0;
  hp.rank_count = ranks;
  hp.ws.status = flags;
  hp.ws.tile_cnt = reinterpret_cast<int32_t*>(static_cast<unsigned char*>(base) + kFlagsBytes);
  hp.ids = dev_topk_ids;
  hp.out_omega = nullptr;
  hp.n_ids = (int)n_ids;
  hp.row_stride = n_ids;
  hp.first_id = 0;
  hp.tile_ids = kStaticTileIds;
  hp.tiles = (int)tiles;
  hp.max_tiles = (int)tiles;
  hp.vec_ok = (n_ids % 4 == 0) && ((reinterpret_cast<uintptr_t>(dev_topk_ids) & 15u) == 0);
  e = launch_hist(hp, batch, 0, stream);
  if (e == cudaSuccess) {
    OmegaParams op = {};   // every rank its own "domain": plain tile sums into dev_omega (bump_serial 0)
    op.d.R = ranks;
    op.d.M = ranks;
    op.d.G = 1;
    op.d.E = experts;
    op.d.sms = sms;
    op.ws.tile_cnt = hp.ws.tile_cnt;
    op.out_omega = dev_omega;
    op.tiles = hp.tiles;
    op.max_tiles = hp.max_tiles;
    op.epw = 32;
    op.rank_first = 0;
    op.rank_count = ranks;
    e = launch_omega(op, batch, stream);
  }
  return e == cudaSuccess ? TOPOEP_OK : TOPOEP_ERR_CUDA;
}

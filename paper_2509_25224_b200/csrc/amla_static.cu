// amla_mla_decode_static: the decode call for callers that must not allocate device memory.
//
// The ordinary entry point takes its scratch (schedule prefix, status word, FP32 partials of split sequences) from a
// workspace the caller allocates.  Some callers cannot do that: code that runs where cudaMalloc is forbidden or
// unaffordable -- inside a latency-critical serving loop that must never touch the allocator, in a process whose
// memory pool was handed out completely at start-up, or in a plugin that is only given input and output buffers.
// For them the same three kernels run here on a scratch area that is part of the library image: a file-scope
// __device__ array of fixed size, present on every GPU that loads the library until the process exits.
#include <atomic>
#include <cstring>

#include "../../include/amla.h"
#include "amla_common.cuh"

#include <mutex>

namespace amla {
int configure_schedule(DecodeParams& prm, int device, int sms, int flags);
int launch_decode_call(const DecodeParams& prm, int* prefix, cudaStream_t stream, int* launches, void (*mark)(int, cudaStream_t));
}  // namespace amla

namespace {

constexpr size_t kAlign = 256;
constexpr size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

constexpr int kMaxItems = AMLA_STATIC_MAX_ITEMS;      // (sequence, 128-row block) pairs
constexpr int kMaxParts = AMLA_STATIC_MAX_SMS / 2;    // clusters

// status | prefix[kMaxItems + 1] | item info [kMaxItems] | partial lse [2 * parts][128] | partial O [2 * parts][128][512]
constexpr size_t kStatusOff = 0;
constexpr size_t kPrefixOff = kAlign;
constexpr size_t kInfoOff = kPrefixOff + align_up(sizeof(int) * (kMaxItems + 1));
constexpr size_t kPartLseOff = kInfoOff + align_up(sizeof(int2) * kMaxItems);
constexpr size_t kPartOOff = kPartLseOff + align_up(sizeof(float) * 2 * kMaxParts * amla::kRowBlock);
constexpr size_t kScratchBytes = kPartOOff + sizeof(float) * 2 * kMaxParts * amla::kRowBlock * amla::kDv;
static_assert(kScratchBytes <= (40u << 20), "the built-in scratch is meant to stay modest");

// The scratch itself.  In host code this name is only a handle for cudaGetSymbolAddress: it is NOT a device address,
// and a kernel handed `g_scratch` directly would fault (or, where the GPU can reach host memory, scribble over the
// wrong bytes).  Host code below always goes through the address looked up per device.
static __device__ __align__(256) unsigned char g_scratch[kScratchBytes];

struct PerDevice {
  std::atomic<int> ready{0};
  std::mutex setup;               // serialises the one-time lookup when first calls race on a device
  unsigned char* scratch = nullptr;
  int sms = 0;
  int cc_major = 0;
};
PerDevice g_dev[64];

// First use on a device (that device being current): look up where this device keeps its copy of the array.
int setup_device(int device, PerDevice** out) {
  if (device < 0 || device >= 64) return AMLA_ERR_INVALID_ARG;
  PerDevice& d = g_dev[device];
  if (!d.ready.load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(d.setup);
    if (d.ready.load(std::memory_order_acquire)) { *out = &d; return AMLA_OK; }
    void* p = nullptr;
    int sms = 0, cc = 0;
    if (cudaGetSymbolAddress(&p, g_scratch) != cudaSuccess || p == nullptr ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&cc, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) {
      cudaGetLastError();
      return AMLA_ERR_CUDA;
    }
    d.scratch = static_cast<unsigned char*>(p);
    d.sms = sms;
    d.cc_major = cc;
    d.ready.store(1, std::memory_order_release);
  }
  *out = &d;
  return AMLA_OK;
}

}  // namespace

extern "C" int amla_mla_decode_static(const void* q, const void* kv_cache, const int32_t* block_table,
                                      const int32_t* seqlens, float softmax_scale, int B, int Sq, int H,
                                      int num_blocks, int max_blocks_per_seq, void* out, float* lse,
                                      void* cuda_stream) {
  using namespace amla;
  if (!q || !kv_cache || !block_table || !seqlens || !out || !lse) return AMLA_ERR_INVALID_ARG;
  if (B <= 0 || Sq <= 0 || H <= 0 || num_blocks <= 0 || max_blocks_per_seq <= 0) return AMLA_ERR_INVALID_ARG;
  if (!(softmax_scale == softmax_scale)) return AMLA_ERR_INVALID_ARG;
  if (Sq > 8 || H > 128) return AMLA_ERR_UNSUPPORTED;
  if (static_cast<long long>(max_blocks_per_seq) * kPage > (1ll << 30)) return AMLA_ERR_UNSUPPORTED;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kv_cache) | reinterpret_cast<uintptr_t>(out)) & 15)
    return AMLA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(block_table) | reinterpret_cast<uintptr_t>(seqlens) | reinterpret_cast<uintptr_t>(lse)) & 3)
    return AMLA_ERR_INVALID_ARG;
  // counted in 128-row blocks, whichever kernel the shape selects
  const long long n_items = static_cast<long long>(B) * ((Sq * H + kRowBlock - 1) / kRowBlock);
  if (n_items > kMaxItems) return AMLA_ERR_STATIC_LIMIT;      // more (sequence, row block) pairs than the scratch has room for

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  PerDevice* dev = nullptr;
  const int rc = setup_device(device, &dev);
  if (rc != AMLA_OK) return rc;
  if (dev->cc_major != 10) return AMLA_ERR_UNSUPPORTED;
  if (dev->sms > AMLA_STATIC_MAX_SMS) return AMLA_ERR_STATIC_LIMIT;   // a device with more SMs than the scratch was sized for

  unsigned char* ws = dev->scratch;
  DecodeParams prm;
  std::memset(&prm, 0, sizeof(prm));
  prm.q = static_cast<const __nv_bfloat16*>(q);
  prm.kv = static_cast<const __nv_bfloat16*>(kv_cache);
  prm.block_table = block_table;
  prm.seqlens = seqlens;
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.lse = lse;
  prm.status = reinterpret_cast<int*>(ws + kStatusOff);
  int* prefix = reinterpret_cast<int*>(ws + kPrefixOff);
  prm.prefix = prefix;
  prm.item_info = reinterpret_cast<int2*>(ws + kInfoOff);
  prm.part_lse = reinterpret_cast<float*>(ws + kPartLseOff);
  prm.part_o = reinterpret_cast<float*>(ws + kPartOOff);
  prm.scale_log2 = softmax_scale * kLog2e;
  prm.out_scale = 1.f;
  prm.B = B; prm.Sq = Sq; prm.H = H;
  prm.R = Sq * H;
  prm.num_blocks = num_blocks;
  prm.max_blocks_per_seq = max_blocks_per_seq;
  prm.flags = AMLA_RESCALE_ALG2 | AMLA_LAZY(AMLA_DEFAULT_TAU);
  prm.tau = static_cast<float>(AMLA_DEFAULT_TAU);
  const int rcfg = configure_schedule(prm, device, dev->sms, prm.flags);
  if (rcfg != AMLA_OK) return rcfg;

  // Nothing in the scratch has to be cleared by the host: the first kernel (the schedule kernel, or for few items the
  // decode kernel itself) rewrites the status word and the whole prefix, and every partial that the combine reads is
  // written by the decode kernel of the same call.
  int launches = 0;
  return launch_decode_call(prm, prefix, static_cast<cudaStream_t>(cuda_stream), &launches, nullptr);
}

extern "C" int amla_static_check_status(void* cuda_stream) {
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  PerDevice* dev = nullptr;
  const int rc = setup_device(device, &dev);
  if (rc != AMLA_OK) return rc;
  int st = 0;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&st, dev->scratch + kStatusOff, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    cudaGetLastError();
    return AMLA_ERR_CUDA;
  }
  return st == amla::kStatusOk ? AMLA_OK : AMLA_ERR_DEVICE_TIMEOUT;
}

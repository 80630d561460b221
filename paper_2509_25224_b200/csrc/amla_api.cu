// C-ABI entry points of libamla: argument validation, workspace carving and the three launches
// (schedule prefix, decode, combine) on the caller's stream.
#include <atomic>
#include <cstring>
#include <new>

#include "../../include/amla.h"
#include "amla_common.cuh"

namespace amla {
cudaError_t launch_plan(const DecodeParams& prm, int* prefix_out, cudaStream_t stream);
cudaError_t launch_combine(const DecodeParams& prm, cudaStream_t stream);
cudaError_t launch_decode_simt(const DecodeParams& prm, cudaStream_t stream);
// Returns cudaSuccess, or an error; sets *unsupported when the device cannot run the kernel.
cudaError_t launch_decode_tc(const DecodeParams& prm, cudaStream_t stream, int* unsupported);
cudaError_t launch_decode_quad(const DecodeParams& prm, cudaStream_t stream, int* unsupported);
cudaError_t launch_wait_selftest(int* status, unsigned long long limit_ns, cudaStream_t stream);
cudaError_t launch_widen_pages(const uint8_t* kv8, const int32_t* block_table, const int32_t* seqlens, int B, int num_blocks,
                               int max_blocks_per_seq, __nv_bfloat16* scratch, int32_t* table_out, cudaStream_t stream);
int decode_tc_parts(int sm_count);
int decode_quad_parts(int device, int sm_count);

namespace {

constexpr size_t kAlign = 256;
constexpr int kMaxRows = 1024;   // Sq * H

size_t align_up(size_t x) { return (x + kAlign - 1) / kAlign * kAlign; }

struct Layout {
  size_t status_off, prefix_off, info_off, part_lse_off, part_o_off, total;
};

Layout make_layout(int n_items, int max_parts) {
  Layout l;
  l.status_off = 0;
  l.prefix_off = kAlign;
  l.info_off = l.prefix_off + align_up(sizeof(int) * (static_cast<size_t>(n_items) + 1));
  l.part_lse_off = l.info_off + align_up(sizeof(int2) * static_cast<size_t>(n_items));
  l.part_o_off = l.part_lse_off + align_up(sizeof(float) * 2 * static_cast<size_t>(max_parts) * kRowBlock);
  l.total = l.part_o_off + sizeof(float) * 2 * static_cast<size_t>(max_parts) * kRowBlock * kDv;
  return l;
}

int check_shape(int B, int Sq, int H, int max_blocks_per_seq) {
  if (B <= 0 || Sq <= 0 || H <= 0 || max_blocks_per_seq <= 0) return AMLA_ERR_INVALID_ARG;
  if (Sq > 8 || H > 128 || Sq * H > kMaxRows) return AMLA_ERR_UNSUPPORTED;
  if (static_cast<long long>(max_blocks_per_seq) * kPage > (1ll << 30)) return AMLA_ERR_UNSUPPORTED;
  if (static_cast<long long>(B) * ((Sq * H + kRowBlock - 1) / kRowBlock) > (1ll << 24)) return AMLA_ERR_UNSUPPORTED;
  return AMLA_OK;
}

// SM count and compute capability per device, queried once (the attributes never change).
constexpr int kMaxDevices = 64;
struct DeviceInfo { std::atomic<int> ready{0}; int sms = 0; int cc_major = 0; };
DeviceInfo g_devices[kMaxDevices];

int sm_count_of(int device, int* sms, int* cc_major) {
  if (device < 0 || device >= kMaxDevices) return AMLA_ERR_INVALID_ARG;
  DeviceInfo& d = g_devices[device];
  if (!d.ready.load(std::memory_order_acquire)) {
    int s = 0, c = 0;
    if (cudaDeviceGetAttribute(&s, cudaDevAttrMultiProcessorCount, device) != cudaSuccess ||
        cudaDeviceGetAttribute(&c, cudaDevAttrComputeCapabilityMajor, device) != cudaSuccess) {
      cudaGetLastError();
      return AMLA_ERR_CUDA;
    }
    d.sms = s; d.cc_major = c;
    d.ready.store(1, std::memory_order_release);
  }
  *sms = d.sms;
  *cc_major = d.cc_major;
  return AMLA_OK;
}

thread_local int g_last_launches = 0;
#ifdef AMLA_TRACE
thread_local unsigned long long* g_trace = nullptr;
#endif

// Optional per-kernel timing (measurement aid): four events bracketing the three launches.
thread_local bool g_profile = false;
thread_local cudaEvent_t g_ev[4] = {nullptr, nullptr, nullptr, nullptr};
thread_local bool g_ev_valid = false;

void profile_mark(int i, cudaStream_t stream) {
  if (g_profile && g_ev[i]) { cudaEventRecord(g_ev[i], stream); if (i == 3) g_ev_valid = true; }
}

}  // namespace

// Chooses the kernel for the shape and fills the schedule fields of prm (rows per item, keys per tile, parts).
// Sequences with more than 128 query rows go to the 256-row kernel (four-CTA clusters, pair MMAs) unless
// AMLA_FLAG_KERNEL_ROWS128 asks for the 128-row kernel.
int configure_schedule(DecodeParams& prm, int device, int sms, int flags) {
  const bool simt = (flags & AMLA_FLAG_KERNEL_SIMT) != 0;
  bool quad = !simt && !(flags & AMLA_FLAG_KERNEL_ROWS128) && prm.R > kRowBlock;
  int quad_parts = 0;
  if (quad) {
    quad_parts = decode_quad_parts(device, sms);
    if (quad_parts <= 0) quad = false;         // four-CTA clusters cannot be placed on this device
  }
  prm.item_rows = quad ? 2 * kRowBlock : kRowBlock;
  prm.tile_keys = quad ? 2 * kPage : kPage;
  prm.ovh = quad ? kQuadOverheadTiles : kUnitOverheadTiles;
  prm.nrb = (prm.R + prm.item_rows - 1) / prm.item_rows;
  prm.n_items = prm.B * prm.nrb;
  prm.P = simt ? sms : quad ? quad_parts : decode_tc_parts(sms);
  prm.fused_plan = (!simt && prm.n_items <= kFusedPlanMaxItems) ? 1 : 0;
  return AMLA_OK;
}

// The launches of one decode call (schedule kernel for large batches, decode, combine) on `stream`.
int launch_decode_call(const DecodeParams& prm, int* prefix, cudaStream_t stream, int* launches, void (*mark)(int, cudaStream_t)) {
  const bool simt = (prm.flags & AMLA_FLAG_KERNEL_SIMT) != 0;
  if (mark) mark(0, stream);
  if (!prm.fused_plan) {
    if (launch_plan(prm, prefix, stream) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
    ++*launches;
  }
  if (mark) mark(1, stream);
  if (simt) {
    if (launch_decode_simt(prm, stream) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  } else {
    int unsupported = 0;
    const cudaError_t err = prm.item_rows > kRowBlock ? launch_decode_quad(prm, stream, &unsupported)
                                                      : launch_decode_tc(prm, stream, &unsupported);
    if (err != cudaSuccess) {
      cudaGetLastError();
      return unsupported ? AMLA_ERR_UNSUPPORTED : AMLA_ERR_CUDA;
    }
  }
  ++*launches;
  if (mark) mark(2, stream);
  if (launch_combine(prm, stream) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  ++*launches;
  if (mark) mark(3, stream);
  return AMLA_OK;
}

}  // namespace amla

using namespace amla;

extern "C" const char* amla_status_string(int status) {
  switch (status) {
    case AMLA_OK: return "ok";
    case AMLA_ERR_INVALID_ARG: return "invalid argument";
    case AMLA_ERR_UNSUPPORTED: return "unsupported shape or device";
    case AMLA_ERR_WORKSPACE: return "workspace too small";
    case AMLA_ERR_CUDA: return "CUDA call failed";
    case AMLA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case AMLA_ERR_STATIC_LIMIT: return "problem or device exceeds the built-in scratch of amla_mla_decode_static";
    default: return "unknown status";
  }
}

extern "C" int amla_mla_decode_workspace_size(int B, int Sq, int H, int max_blocks_per_seq, int device,
                                              size_t* bytes_out) {
  if (!bytes_out) return AMLA_ERR_INVALID_ARG;
  int rc = check_shape(B, Sq, H, max_blocks_per_seq);
  if (rc != AMLA_OK) return rc;
  int sms = 0, cc = 0;
  rc = sm_count_of(device, &sms, &cc);
  if (rc != AMLA_OK) return rc;
  const int nrb = (Sq * H + kRowBlock - 1) / kRowBlock;
  *bytes_out = make_layout(B * nrb, sms).total;
  return AMLA_OK;
}

namespace {

// The decode call on a bf16 cache.  out_scale multiplies the normalised output (1 unless the cache was widened from
// FP8 with a dequantisation scale); launches are added to g_last_launches.
int decode_impl(const void* q, const void* kv_cache, const int32_t* block_table, const int32_t* seqlens,
                float softmax_scale, float out_scale, int B, int Sq, int H, int num_blocks, int max_blocks_per_seq,
                void* out, float* lse, void* workspace, size_t workspace_bytes, void* cuda_stream, int flags) {
  if (!q || !kv_cache || !block_table || !seqlens || !out || !lse || !workspace) return AMLA_ERR_INVALID_ARG;
  if (num_blocks <= 0 || !(softmax_scale == softmax_scale)) return AMLA_ERR_INVALID_ARG;
  int rc = check_shape(B, Sq, H, max_blocks_per_seq);
  if (rc != AMLA_OK) return rc;
  if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(kv_cache) | reinterpret_cast<uintptr_t>(out)) & 15)
    return AMLA_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(block_table) | reinterpret_cast<uintptr_t>(seqlens) | reinterpret_cast<uintptr_t>(lse)) & 3)
    return AMLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) return AMLA_ERR_INVALID_ARG;
  if ((flags & AMLA_RESCALE_MASK) == 3) return AMLA_ERR_INVALID_ARG;

  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  int sms = 0, cc = 0;
  rc = sm_count_of(device, &sms, &cc);
  if (rc != AMLA_OK) return rc;
  if (cc != 10) return AMLA_ERR_UNSUPPORTED;

  // the layout is sized for 128-row items (the larger item count) whichever kernel runs
  const Layout lay = make_layout(B * ((Sq * H + kRowBlock - 1) / kRowBlock), sms);
  if (workspace_bytes < lay.total) return AMLA_ERR_WORKSPACE;

  char* ws = static_cast<char*>(workspace);
  DecodeParams prm;
  std::memset(&prm, 0, sizeof(prm));
  prm.q = static_cast<const __nv_bfloat16*>(q);
  prm.kv = static_cast<const __nv_bfloat16*>(kv_cache);
  prm.block_table = block_table;
  prm.seqlens = seqlens;
  prm.out = static_cast<__nv_bfloat16*>(out);
  prm.lse = lse;
  prm.status = reinterpret_cast<int*>(ws + lay.status_off);
  int* prefix = reinterpret_cast<int*>(ws + lay.prefix_off);
  prm.prefix = prefix;
  prm.item_info = reinterpret_cast<int2*>(ws + lay.info_off);
  prm.part_lse = reinterpret_cast<float*>(ws + lay.part_lse_off);
  prm.part_o = reinterpret_cast<float*>(ws + lay.part_o_off);
  prm.scale_log2 = softmax_scale * kLog2e;
  prm.out_scale = out_scale;
  prm.B = B; prm.Sq = Sq; prm.H = H;
  prm.R = Sq * H;
  prm.num_blocks = num_blocks;
  prm.max_blocks_per_seq = max_blocks_per_seq;
  prm.flags = flags;
#ifdef AMLA_TRACE
  prm.trace = g_trace;
#endif
  prm.tau = static_cast<float>((flags & AMLA_LAZY_MASK) >> AMLA_LAZY_SHIFT);
  rc = configure_schedule(prm, device, sms, flags);
  if (rc != AMLA_OK) return rc;
  return launch_decode_call(prm, prefix, static_cast<cudaStream_t>(cuda_stream), &g_last_launches, profile_mark);
}

// Bytes of the FP8 path's extra scratch behind the ordinary workspace: the new block table and the widened pages.
size_t fp8_table_bytes(int B, int max_blocks_per_seq) { return align_up(sizeof(int32_t) * static_cast<size_t>(B) * max_blocks_per_seq); }
size_t fp8_pages_bytes(int B, int max_blocks_per_seq) { return static_cast<size_t>(B) * max_blocks_per_seq * kPage * kDqk * sizeof(__nv_bfloat16); }

}  // namespace

extern "C" int amla_mla_decode_ex(const void* q, const void* kv_cache, const int32_t* block_table,
                                  const int32_t* seqlens, float softmax_scale, int B, int Sq, int H,
                                  int num_blocks, int max_blocks_per_seq, void* out, float* lse,
                                  void* workspace, size_t workspace_bytes, void* cuda_stream, int flags) {
  g_last_launches = 0;
  return decode_impl(q, kv_cache, block_table, seqlens, softmax_scale, 1.f, B, Sq, H, num_blocks, max_blocks_per_seq, out, lse,
                     workspace, workspace_bytes, cuda_stream, flags);
}

extern "C" int amla_mla_decode_fp8_workspace_size(int B, int Sq, int H, int max_blocks_per_seq, int device, size_t* bytes_out) {
  size_t base = 0;
  const int rc = amla_mla_decode_workspace_size(B, Sq, H, max_blocks_per_seq, device, &base);
  if (rc != AMLA_OK) return rc;
  *bytes_out = align_up(base) + fp8_table_bytes(B, max_blocks_per_seq) + fp8_pages_bytes(B, max_blocks_per_seq);
  return AMLA_OK;
}

extern "C" int amla_mla_decode_fp8(const void* q, const void* kv_cache_e4m3, float kv_scale, const int32_t* block_table,
                                   const int32_t* seqlens, float softmax_scale, int B, int Sq, int H, int num_blocks,
                                   int max_blocks_per_seq, void* out, float* lse, void* workspace, size_t workspace_bytes,
                                   void* cuda_stream, int flags) {
  g_last_launches = 0;
  if (!q || !kv_cache_e4m3 || !block_table || !seqlens || !out || !lse || !workspace) return AMLA_ERR_INVALID_ARG;
  if (num_blocks <= 0 || !(kv_scale == kv_scale) || !(softmax_scale == softmax_scale)) return AMLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(kv_cache_e4m3) & 15) return AMLA_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) return AMLA_ERR_INVALID_ARG;
  int rc = check_shape(B, Sq, H, max_blocks_per_seq);
  if (rc != AMLA_OK) return rc;
  int device = 0;
  if (cudaGetDevice(&device) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  size_t base = 0;
  rc = amla_mla_decode_workspace_size(B, Sq, H, max_blocks_per_seq, device, &base);
  if (rc != AMLA_OK) return rc;
  base = align_up(base);
  const size_t tbytes = fp8_table_bytes(B, max_blocks_per_seq), pbytes = fp8_pages_bytes(B, max_blocks_per_seq);
  if (workspace_bytes < base + tbytes + pbytes) return AMLA_ERR_WORKSPACE;
  if (static_cast<long long>(B) * max_blocks_per_seq > (1ll << 30)) return AMLA_ERR_UNSUPPORTED;
  char* ws = static_cast<char*>(workspace);
  int32_t* table2 = reinterpret_cast<int32_t*>(ws + base);
  __nv_bfloat16* pages = reinterpret_cast<__nv_bfloat16*>(ws + base + tbytes);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (launch_widen_pages(static_cast<const uint8_t*>(kv_cache_e4m3), block_table, seqlens, B, num_blocks, max_blocks_per_seq,
                         pages, table2, stream) != cudaSuccess) {
    cudaGetLastError();
    return AMLA_ERR_CUDA;
  }
  ++g_last_launches;
  // logits: scale * q . (k8 * kv_scale); output: sum p * (v8 * kv_scale)
  return decode_impl(q, pages, table2, seqlens, softmax_scale * kv_scale, kv_scale, B, Sq, H, B * max_blocks_per_seq,
                     max_blocks_per_seq, out, lse, workspace, base, cuda_stream, flags);
}

extern "C" int amla_mla_decode(const void* q, const void* kv_cache, const int32_t* block_table,
                               const int32_t* seqlens, float softmax_scale, int B, int Sq, int H,
                               int num_blocks, int max_blocks_per_seq, void* out, float* lse,
                               void* workspace, size_t workspace_bytes, void* cuda_stream) {
  return amla_mla_decode_ex(q, kv_cache, block_table, seqlens, softmax_scale, B, Sq, H, num_blocks,
                            max_blocks_per_seq, out, lse, workspace, workspace_bytes, cuda_stream,
                            AMLA_RESCALE_ALG2 | AMLA_LAZY(AMLA_DEFAULT_TAU));
}

extern "C" int amla_check_status(const void* workspace, void* cuda_stream) {
  if (!workspace) return AMLA_ERR_INVALID_ARG;
  int st = 0;
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  if (cudaMemcpyAsync(&st, workspace, sizeof(int), cudaMemcpyDeviceToHost, stream) != cudaSuccess ||
      cudaStreamSynchronize(stream) != cudaSuccess) {
    cudaGetLastError();
    return AMLA_ERR_CUDA;
  }
  return st == kStatusOk ? AMLA_OK : AMLA_ERR_DEVICE_TIMEOUT;
}

extern "C" int amla_last_launch_count(void) { return g_last_launches; }

extern "C" int amla_wait_selftest(void* workspace, unsigned long long limit_ns, void* cuda_stream) {
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 3)) return AMLA_ERR_INVALID_ARG;
  if (limit_ns == 0 || limit_ns > 100000000ull) return AMLA_ERR_INVALID_ARG;      // at most 0.1 s
  if (launch_wait_selftest(static_cast<int*>(workspace), limit_ns, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess) {
    cudaGetLastError();
    return AMLA_ERR_CUDA;
  }
  return AMLA_OK;
}

extern "C" int amla_validate_paging_host(const int32_t* block_table, const int32_t* seqlens, int B, int num_blocks,
                                         int max_blocks_per_seq, int* bad_seq, int* bad_block) {
  if (!block_table || !seqlens || B <= 0 || num_blocks <= 0 || max_blocks_per_seq <= 0) return AMLA_ERR_INVALID_ARG;
  for (int b = 0; b < B; ++b) {
    const long long n = seqlens[b];
    if (n < 0 || n > static_cast<long long>(max_blocks_per_seq) * kPage) {
      if (bad_seq) *bad_seq = b;
      if (bad_block) *bad_block = -1;
      return AMLA_ERR_INVALID_ARG;
    }
    const int used = static_cast<int>((n + kPage - 1) / kPage);
    for (int i = 0; i < used; ++i) {
      const int32_t pg = block_table[static_cast<size_t>(b) * max_blocks_per_seq + i];
      if (pg < 0 || pg >= num_blocks) {
        if (bad_seq) *bad_seq = b;
        if (bad_block) *bad_block = i;
        return AMLA_ERR_INVALID_ARG;
      }
    }
  }
  return AMLA_OK;
}

extern "C" int amla_profile_enable(int on) {
  if (on && !g_ev[0]) {
    for (int i = 0; i < 4; ++i) {
      if (cudaEventCreate(&g_ev[i]) != cudaSuccess) { cudaGetLastError(); g_ev[i] = nullptr; return AMLA_ERR_CUDA; }
    }
  }
  g_profile = on != 0;
  g_ev_valid = false;
  return AMLA_OK;
}

extern "C" int amla_profile_last_ms(float* ms3) {
  if (!ms3) return AMLA_ERR_INVALID_ARG;
  if (!g_ev_valid) return AMLA_ERR_INVALID_ARG;
  if (cudaEventSynchronize(g_ev[3]) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  for (int i = 0; i < 3; ++i) {
    if (cudaEventElapsedTime(&ms3[i], g_ev[i], g_ev[i + 1]) != cudaSuccess) { cudaGetLastError(); return AMLA_ERR_CUDA; }
  }
  return AMLA_OK;
}

extern "C" int amla_plan_host(const int32_t* seqlens, int B, int Sq, int H, int num_parts, int32_t* units,
                              int max_units) {
  if (!seqlens || !units || num_parts <= 0 || max_units < 0) return AMLA_ERR_INVALID_ARG;
  int rc = check_shape(B, Sq, H, 1);
  if (rc != AMLA_OK) return rc;
  const bool quad = Sq * H > kRowBlock;
  const int item_rows = quad ? 2 * kRowBlock : kRowBlock, tile_keys = quad ? 2 * kPage : kPage;
  const int ovh = quad ? kQuadOverheadTiles : kUnitOverheadTiles;
  const int nrb = (Sq * H + item_rows - 1) / item_rows;
  const int n_items = B * nrb;
  int* prefix = new (std::nothrow) int[n_items + 1];
  if (!prefix) return AMLA_ERR_WORKSPACE;
  int acc = 0;
  for (int it = 0; it < n_items; ++it) {
    prefix[it] = acc;
    acc += schedule_length(seqlens[it / nrb], it, tile_keys, ovh);
  }
  prefix[n_items] = acc;
  const Plan plan = Plan::make(prefix, n_items, num_parts, ovh);
  int n_units = 0;
  bool overflow = false;
  if (acc > 0) {
    for (int p = 0; p < plan.P; ++p) {
      const int g0 = plan.part_start(p), g1 = plan.part_start(p + 1);
      int g = g0;
      while (g < g1) {
        const int it = plan.item_of_tile(g);
        const int a = plan.first_tile(it), e = prefix[it + 1];
        const int lo = g > a ? g : a, hi = e < g1 ? e : g1;
        g = e < g1 ? e : g1;
        if (hi <= lo) continue;
        const int t0 = lo - a, t1 = hi - a;
        int p_first, p_last;
        const int nsplit = plan.item_parts(it, &p_first, &p_last);
        if (n_units < max_units) {
          int32_t* u = units + 6 * n_units;
          u[0] = p; u[1] = it; u[2] = t0; u[3] = t1;
          u[4] = nsplit == 1 ? -1 : plan.slot_of(p, it, p_first);
          u[5] = nsplit;
        } else {
          overflow = true;
        }
        ++n_units;
      }
    }
  }
  delete[] prefix;
  return overflow ? AMLA_ERR_WORKSPACE : n_units;
}

#ifdef AMLA_TRACE
// Trace builds only (not part of the public header): device buffer of
// parts * kTraceEvents * kTraceTiles 64-bit stamps that later calls on this thread fill.
extern "C" int amla_debug_set_trace(void* device_buffer) {
  g_trace = static_cast<unsigned long long*>(device_buffer);
  return AMLA_OK;
}
#endif

// Split-KV schedule (prefix of tile counts per work item) and the lse-weighted combine of split
// partials.  Neither is in the paper: its kernel runs batch 96 on 48 cores, whereas a decode batch
// here has far fewer (sequence, row-block) items than the GPU has SMs.  The combine is the
// log-sum-exp merge that follows from the blockwise associativity of Algorithm 1's recurrence.
#include "amla_common.cuh"

namespace amla {

// One block.  prefix[it] = sum over items before `it` of their schedule lengths (tiles plus the start-up
// overhead of a non-empty item, see Plan); also resets the
// status word.  n_items is small (B * ceil(Sq*H/128)); a chunked block scan covers any size.
__global__ void plan_kernel(const int32_t* __restrict__ seqlens, int nrb, int n_items, int tile_keys, int ovh,
                            int* __restrict__ prefix, int* __restrict__ status) {
  __shared__ int warp_sums[32];
  __shared__ int carry;
  asm volatile("griddepcontrol.launch_dependents;");   // the decode kernel may start its set-up; it waits before reading
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  if (tid == 0) { carry = 0; *status = kStatusOk; }
  __syncthreads();
  for (int base = 0; base < n_items; base += blockDim.x) {
    const int it = base + tid;
    int v = 0;
    if (it < n_items) v = schedule_length(seqlens[it / nrb], it, tile_keys, ovh);
    int x = v;  // inclusive warp scan
    for (int o = 1; o < 32; o <<= 1) {
      int y = __shfl_up_sync(0xffffffffu, x, o);
      if (lane >= o) x += y;
    }
    if (lane == 31) warp_sums[wid] = x;
    __syncthreads();
    if (wid == 0) {
      int s = (lane < (blockDim.x >> 5)) ? warp_sums[lane] : 0;
      for (int o = 1; o < 32; o <<= 1) {
        int y = __shfl_up_sync(0xffffffffu, s, o);
        if (lane >= o) s += y;
      }
      warp_sums[lane] = s;  // inclusive over warps
    }
    __syncthreads();
    const int before = carry + (wid ? warp_sums[wid - 1] : 0) + (x - v);
    if (it < n_items) prefix[it] = before;
    __syncthreads();
    if (tid == blockDim.x - 1) carry = before + v;
    __syncthreads();
  }
  if (tid == 0) prefix[n_items] = carry;
}

// One warp per query row.  Items that one part covered entirely were written by the decode kernel and are skipped;
// items without tiles get out = 0, lse = -inf; split items are merged:
//   lse = ln sum_s exp(lse_s),  out = sum_s exp(lse_s - lse) * out_s.
// What the row needs to know about its item (where its partials are) was left in item_info by the decode kernel, so
// the warp's chain of dependent memory round trips is short: (prefix, item_info) -> (partial lse, partial rows).
// Up to kFastSplits partials are fetched before any arithmetic.
constexpr int kFastSplits = 4;

__global__ void __launch_bounds__(128) combine_kernel(DecodeParams prm) {
#ifdef AMLA_TRACE
  unsigned long long t_ns;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_ns));
  if (prm.trace && blockIdx.x == 0 && threadIdx.x == 0) prm.trace[148 * 16 * 128 + 0] = t_ns & 0xffffffffull;
#endif
  // A decode kernel that follows on the stream may set itself up beside this kernel (it writes nothing this kernel
  // reads before its own wait for this kernel's completion).
  asm volatile("griddepcontrol.launch_dependents;");
  const int warps_per_block = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  const int row_global = blockIdx.x * warps_per_block + (threadIdx.x >> 5);
  const int rows_padded = prm.nrb * prm.item_rows;
  const int b = row_global / rows_padded;
  const int rin = row_global - b * rows_padded;   // row within the sequence, padded to items
  const bool live = b < prm.B && rin < prm.R;
  const int rb = rin / prm.item_rows, rr = rin % prm.item_rows;   // item of the sequence, row within the item
  const int it = b * prm.nrb + rb;
  asm volatile("griddepcontrol.wait;" ::: "memory");   // launched early (programmatic dependent launch): the partials must be complete
#ifdef AMLA_TRACE
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_ns));
  if (prm.trace && blockIdx.x == 0 && threadIdx.x == 0) prm.trace[148 * 16 * 128 + 1] = t_ns & 0xffffffffull;
  if (prm.trace && blockIdx.x == gridDim.x - 1 && threadIdx.x == 0) prm.trace[148 * 16 * 128 + 2] = t_ns & 0xffffffffull;
#endif
  if (!live) return;

  const int pa = prm.prefix[it], pe = prm.prefix[it + 1];
  const int2 info = prm.item_info[it];           // valid only for items with tiles
  __nv_bfloat16* orow = prm.out + (static_cast<size_t>(b) * prm.R + rin) * kDv;
  float* lrow = prm.lse + static_cast<size_t>(b) * prm.R + rin;
  auto write_empty = [&]() {
    for (int c = lane * 8; c < kDv; c += 32 * 8) *reinterpret_cast<uint4*>(orow + c) = make_uint4(0, 0, 0, 0);
    if (lane == 0) *lrow = -INFINITY;
  };
  if (pe <= pa) { write_empty(); return; }       // no tiles: no part ever saw this item
  const int nsplit = info.y;
  if (nsplit == 1) return;

  // a lane merges 16 consecutive columns (half of a 32-column chunk: one scale byte per split)
  const uint16_t* halves = partial_halves(prm);
  const uint8_t* scales = partial_scales(prm);
  float acc[16];
  float tot = 0.f, mx;
  auto accumulate = [&](float w, uint32_t scale_byte, const uint4& a, const uint4& b) {
    const float ws = w * partial_unscale(scale_byte);
    const uint32_t h[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const float2 v = unpack_f16x2(h[i]);
      acc[2 * i] += ws * v.x;
      acc[2 * i + 1] += ws * v.y;
    }
  };
  if (nsplit <= kFastSplits) {
    // everything is requested before anything is used
    float ls[kFastSplits];
    uint4 va[kFastSplits], vb[kFastSplits];
    uint32_t sc[kFastSplits];
#pragma unroll
    for (int s = 0; s < kFastSplits; ++s) {
      ls[s] = -INFINITY;
      if (s < nsplit) {
        const size_t prow = static_cast<size_t>(Plan::slot_of_split(info.x, s)) * prm.item_rows + rr;
        ls[s] = prm.part_lse[prow];
        sc[s] = scales[prow * 16 + (lane >> 1)];
        const uint4* src = reinterpret_cast<const uint4*>(halves + prow * kDv) + 2 * lane;
        va[s] = src[0];
        vb[s] = src[1];
      }
    }
    mx = ls[0];
#pragma unroll
    for (int s = 1; s < kFastSplits; ++s) mx = fmaxf(mx, ls[s]);
    if (mx == -INFINITY) { write_empty(); return; }   // no split saw a visible key for this row
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
#pragma unroll
    for (int s = 0; s < kFastSplits; ++s) {
      if (s < nsplit) {
        const float w = expf(ls[s] - mx);             // 0 for a split that saw nothing
        tot += w;
        accumulate(w, sc[s], va[s], vb[s]);
      }
    }
  } else {
    // lse of the splits: one split per lane (in rounds of 32), so that the loads overlap
    mx = -INFINITY;
    for (int base = 0; base < nsplit; base += 32) {
      const int sidx = base + lane;
      if (sidx < nsplit) mx = fmaxf(mx, prm.part_lse[static_cast<size_t>(Plan::slot_of_split(info.x, sidx)) * prm.item_rows + rr]);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (mx == -INFINITY) { write_empty(); return; }
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    for (int base = 0; base < nsplit; base += 32) {
      const int sidx = base + lane;
      int my_slot = 0;
      float my_w = 0.f;
      if (sidx < nsplit) {
        my_slot = Plan::slot_of_split(info.x, sidx);
        my_w = expf(prm.part_lse[static_cast<size_t>(my_slot) * prm.item_rows + rr] - mx);
      }
      const int n_here = min(32, nsplit - base);
#pragma unroll 2
      for (int j = 0; j < n_here; ++j) {
        const float w = __shfl_sync(0xffffffffu, my_w, j);
        const int slot = __shfl_sync(0xffffffffu, my_slot, j);
        tot += w;
        const size_t prow = static_cast<size_t>(slot) * prm.item_rows + rr;
        const uint4* src = reinterpret_cast<const uint4*>(halves + prow * kDv) + 2 * lane;
        accumulate(w, scales[prow * 16 + (lane >> 1)], src[0], src[1]);
      }
    }
  }
  const float inv = 1.f / tot;
  uint32_t pk[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    __nv_bfloat162 v = __floats2bfloat162_rn(acc[2 * i] * inv, acc[2 * i + 1] * inv);
    pk[i] = *reinterpret_cast<uint32_t*>(&v);
  }
  uint4* dst = reinterpret_cast<uint4*>(orow + 16 * lane);
  dst[0] = make_uint4(pk[0], pk[1], pk[2], pk[3]);
  dst[1] = make_uint4(pk[4], pk[5], pk[6], pk[7]);
  if (lane == 0) *lrow = mx + logf(tot);
#ifdef AMLA_TRACE
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t_ns));
  if (prm.trace && lane == 0) atomicMax(prm.trace + 148 * 16 * 128 + 3, t_ns & 0xffffffffull);
#endif
}

cudaError_t launch_plan(const DecodeParams& prm, int* prefix_out, cudaStream_t stream) {
  plan_kernel<<<1, 1024, 0, stream>>>(prm.seqlens, prm.nrb, prm.n_items, prm.tile_keys, prm.ovh, prefix_out, prm.status);
  return cudaGetLastError();
}

cudaError_t launch_combine(const DecodeParams& prm, cudaStream_t stream) {
  const int warps_per_block = 4;   // small blocks: one fits beside a decode CTA (registers), so part of the grid is resident before the decode kernel ends
  const long rows = static_cast<long>(prm.B) * prm.nrb * prm.item_rows;
  const int blocks = static_cast<int>((rows + warps_per_block - 1) / warps_per_block);
  // programmatic dependent launch: the blocks may be placed while the decode kernel drains; they wait inside
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(blocks);
  cfg.blockDim = dim3(warps_per_block * 32);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, combine_kernel, prm);
}

}  // namespace amla

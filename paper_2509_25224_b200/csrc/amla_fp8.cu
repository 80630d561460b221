// FP8 (E4M3) latent cache: widening of the pages a batch uses into a bf16 scratch cache, ahead of the decode kernels.
//
// The paper's remark after Lemma 3.1 notes that the exponent-add applies to other floating-point formats; what it
// acts on here stays the FP32 accumulator.  An FP8 cache changes the inputs only: every cache byte is an OCP E4M3
// number (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no infinities, S.1111.111 = NaN) and the stored
// value is byte_value * kv_scale.  E4M3 values are exactly representable in bf16, so the pages are widened without
// rounding, the per-tensor scale is folded into the softmax scale (for the logits) and into the final
// normalisation (for V), and the bf16 kernels run unchanged on the widened copy.  This is a two-pass path: the
// cache occupies half the memory, but a call reads the FP8 pages once and writes and reads their bf16 copy.
#include "amla_common.cuh"

namespace amla {

namespace {

// Two E4M3 bytes (low 16 bits of `pair`) -> two bf16 in one word.  E4M3 -> f16 is one hardware conversion and
// exact; f16 -> f32 -> bf16 is exact for these values (at most four significant bits, exponents -9 .. 8).
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint32_t pair) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(static_cast<unsigned short>(pair & 0xffffu)));
  float lo, hi;
  asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}" : "=f"(lo), "=f"(hi) : "r"(h2));
  uint32_t r;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}

constexpr int kWidenThreads = 256;
constexpr int kPageBytes8 = kPage * kDqk;            // 36 864 bytes of E4M3 per page

}  // namespace

// One block per (sequence, page slot).  Page slot i of sequence b is widened into scratch page b * max_blocks + i
// (and that index is written to the new block table) if the sequence reaches it; a page index outside the cache
// gives a page of zeros.
__global__ void __launch_bounds__(kWidenThreads) widen_pages_kernel(const uint8_t* __restrict__ kv8, const int32_t* __restrict__ block_table,
                                                                    const int32_t* __restrict__ seqlens, int num_blocks, int max_blocks_per_seq,
                                                                    __nv_bfloat16* __restrict__ scratch, int32_t* __restrict__ table_out) {
  asm volatile("griddepcontrol.launch_dependents;");   // the decode kernel may set itself up; it waits before it reads
  const int b = blockIdx.x / max_blocks_per_seq, i = blockIdx.x % max_blocks_per_seq;
  if (threadIdx.x == 0) table_out[blockIdx.x] = blockIdx.x;
  const int n = min(max(seqlens[b], 0), max_blocks_per_seq * kPage);
  if (i * kPage >= n) return;
  const int32_t page = block_table[blockIdx.x];
  const bool in_range = page >= 0 && page < num_blocks;
  const uint4* src = reinterpret_cast<const uint4*>(kv8 + static_cast<size_t>(in_range ? page : 0) * kPageBytes8);
  uint4* dst = reinterpret_cast<uint4*>(scratch + static_cast<size_t>(blockIdx.x) * kPage * kDqk);
  for (int c = threadIdx.x; c < kPageBytes8 / 16; c += kWidenThreads) {
    uint4 x = in_range ? __ldg(src + c) : make_uint4(0, 0, 0, 0);
    uint4 lo, hi;
    lo.x = e4m3x2_to_bf16x2(x.x); lo.y = e4m3x2_to_bf16x2(x.x >> 16);
    lo.z = e4m3x2_to_bf16x2(x.y); lo.w = e4m3x2_to_bf16x2(x.y >> 16);
    hi.x = e4m3x2_to_bf16x2(x.z); hi.y = e4m3x2_to_bf16x2(x.z >> 16);
    hi.z = e4m3x2_to_bf16x2(x.w); hi.w = e4m3x2_to_bf16x2(x.w >> 16);
    dst[2 * c] = lo;
    dst[2 * c + 1] = hi;
  }
}

cudaError_t launch_widen_pages(const uint8_t* kv8, const int32_t* block_table, const int32_t* seqlens, int B, int num_blocks,
                               int max_blocks_per_seq, __nv_bfloat16* scratch, int32_t* table_out, cudaStream_t stream) {
  widen_pages_kernel<<<B * max_blocks_per_seq, kWidenThreads, 0, stream>>>(kv8, block_table, seqlens, num_blocks, max_blocks_per_seq,
                                                                           scratch, table_out);
  return cudaGetLastError();
}

}  // namespace amla

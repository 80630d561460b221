// Line 20 of Algorithm 2 for one 32-column chunk of one row: the accumulator words as they come from tensor memory,
// times 1 / (l * S16), packed for the store (include after amla_common.cuh and amla_sm100.cuh).  The arithmetic is kept short on purpose: the epilogue runs with one or two warps per
// scheduler and nothing to hide a dependent chain behind.
#pragma once

namespace amla {

// Final output: bf16(O * inv), two elements per multiply.
__device__ __forceinline__ void epilogue_chunk_bf16(const uint32_t (&o)[32], float inv, uint32_t (&w)[16]) {
  const uint64_t s2 = sm100::pack_f32x2(inv, inv);
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float a, b;
    sm100::unpack_f32x2(sm100::mul_f32x2(sm100::pack_f32x2(__uint_as_float(o[2 * j]), __uint_as_float(o[2 * j + 1])), s2), a, b);
    w[j] = sm100::pack_bf16x2(a, b);
  }
}

// Split partial: fp16(O * inv * f) with f = the power of two that brings the chunk's largest magnitude below 2;
// returns the chunk's scale byte.  Rounding is monotonic, so max |O * inv| is (max |O|) * inv, and f is a power of
// two, so (O * inv) * f and O * (inv * f) round to the same value: one multiply per element, and the maximum is
// taken on the raw words, three per instruction and on two chains.
__device__ __forceinline__ uint32_t epilogue_chunk_partial(const uint32_t (&o)[32], float inv, uint32_t (&w)[16]) {
  float m0 = sm100::fmax3_abs(__uint_as_float(o[0]), __uint_as_float(o[1]), __uint_as_float(o[2]));
  float m1 = sm100::fmax3_abs(__uint_as_float(o[3]), __uint_as_float(o[4]), __uint_as_float(o[5]));
#pragma unroll
  for (int i = 6; i + 3 < 32; i += 4) {
    m0 = sm100::fmax3_abs(m0, __uint_as_float(o[i]), __uint_as_float(o[i + 1]));
    m1 = sm100::fmax3_abs(m1, __uint_as_float(o[i + 2]), __uint_as_float(o[i + 3]));
  }
  m0 = sm100::fmax3_abs(m0, __uint_as_float(o[30]), __uint_as_float(o[31]));
  float f;
  const uint32_t sb = partial_scale_byte(fmaxf(m0, m1) * fabsf(inv), &f);
  const float g = inv * f;
  const uint64_t s2 = sm100::pack_f32x2(g, g);
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    float a, b;
    sm100::unpack_f32x2(sm100::mul_f32x2(sm100::pack_f32x2(__uint_as_float(o[2 * j]), __uint_as_float(o[2 * j + 1])), s2), a, b);
    w[j] = pack_f16x2(a, b);
  }
  return sb;
}

}  // namespace amla

// TEST INFRASTRUCTURE -- not part of the product path.
//
// FP64 oracle for paged MLA decode attention on an FP8 (OCP E4M3) latent cache: the same plain definition as
// mla_decode_oracle.cpp (Eq. 1 with the MLA sharing of Section 2.2), with every cache byte widened exactly to
// double by the format's definition and multiplied by the per-tensor dequantisation scale:
//
//   byte = S EEEE MMM;  E = 0:        (-1)^S * 2^-6 * (M / 8)
//                       E = 1..15:    (-1)^S * 2^(E-7) * (1 + M / 8)      (S.1111.111 is NaN; there are no infinities)
//   k_j[d] = value(byte) * kv_scale
//   s_j = scale * sum_d q[d] * k_j[d];  m = max_j s_j;  l = sum_j exp(s_j - m)
//   out = sum_j exp(s_j - m) * k_j[0:512] / l;  lse = m + ln(l)
//
// q is bf16 (bit patterns widened exactly).  Visibility rule and empty rows as in mla_decode_oracle.cpp.  No code is
// shared with the CUDA path.  Pins (tests/test_oracle_pins.py): all 256 byte values against a hand-written table of
// the format, and equality with the bf16 oracle on a cache whose bf16 values are the widened bytes.

#include <cmath>
#include <cstdint>
#include <cstring>
#include <limits>
#include <vector>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

constexpr int kDqk = 576;
constexpr int kDv = 512;
constexpr int kPage = 64;

inline double bf16_bits_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof(f));
  return static_cast<double>(f);
}

inline double e4m3_value(uint8_t byte) {
  const int s = byte >> 7, e = (byte >> 3) & 15, m = byte & 7;
  if (e == 15 && m == 7) return std::numeric_limits<double>::quiet_NaN();
  const double mag = e == 0 ? std::ldexp(static_cast<double>(m) / 8.0, -6) : std::ldexp(1.0 + static_cast<double>(m) / 8.0, e - 7);
  return s ? -mag : mag;
}

int one_row_fp8(const uint16_t* q, const uint8_t* kv, double kv_scale, const int32_t* block_table, const int32_t* seqlens,
                double scale, int Sq, int H, int num_blocks, int max_blocks_per_seq, int b, int t, int h, double* out,
                double* lse) {
  const long n_b = seqlens[b];
  long visible = n_b - Sq + t + 1;
  if (visible > n_b) visible = n_b;
  for (int d = 0; d < kDv; ++d) out[d] = 0.0;
  if (visible <= 0) {
    *lse = -std::numeric_limits<double>::infinity();
    return 0;
  }
  const uint16_t* qrow = q + ((static_cast<size_t>(b) * Sq + t) * H + h) * kDqk;
  double qd[kDqk];
  for (int d = 0; d < kDqk; ++d) qd[d] = bf16_bits_to_double(qrow[d]);
  std::vector<double> s(static_cast<size_t>(visible));
  double m = -std::numeric_limits<double>::infinity();
  for (long j = 0; j < visible; ++j) {
    const long blk = j / kPage;
    if (blk >= max_blocks_per_seq) return 1;
    const int32_t page = block_table[static_cast<size_t>(b) * max_blocks_per_seq + blk];
    if (page < 0 || page >= num_blocks) return 1;
    const uint8_t* krow = kv + (static_cast<size_t>(page) * kPage + (j % kPage)) * kDqk;
    double acc = 0.0;
    for (int d = 0; d < kDqk; ++d) acc += qd[d] * (e4m3_value(krow[d]) * kv_scale);
    s[j] = acc * scale;
    if (s[j] > m) m = s[j];
  }
  double l = 0.0;
  for (long j = 0; j < visible; ++j) {
    const double p = std::exp(s[j] - m);
    l += p;
    const int32_t page = block_table[static_cast<size_t>(b) * max_blocks_per_seq + j / kPage];
    const uint8_t* krow = kv + (static_cast<size_t>(page) * kPage + (j % kPage)) * kDqk;
    for (int d = 0; d < kDv; ++d) out[d] += p * (e4m3_value(krow[d]) * kv_scale);
  }
  for (int d = 0; d < kDv; ++d) out[d] /= l;
  *lse = m + std::log(l);
  return 0;
}

}  // namespace

extern "C" {

// The widening alone (for its pin).
double oracle_e4m3_to_double(uint8_t byte) { return e4m3_value(byte); }

// Full problem on an E4M3 cache.  out: double [B, Sq, H, 512]; lse: double [B, Sq, H].
int oracle_mla_decode_fp8(const uint16_t* q, const uint8_t* kv, double kv_scale, const int32_t* block_table,
                          const int32_t* seqlens, double scale, int B, int Sq, int H, int num_blocks,
                          int max_blocks_per_seq, double* out, double* lse, int n_threads) {
  int bad = 0;
  const long rows = static_cast<long>(B) * Sq * H;
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel for schedule(dynamic, 1) reduction(| : bad)
  for (long r = 0; r < rows; ++r) {
    const int h = static_cast<int>(r % H);
    const int t = static_cast<int>((r / H) % Sq);
    const int b = static_cast<int>(r / (static_cast<long>(H) * Sq));
    bad |= one_row_fp8(q, kv, kv_scale, block_table, seqlens, scale, Sq, H, num_blocks, max_blocks_per_seq, b, t, h,
                       out + r * kDv, lse + r);
  }
  return bad;
}

}  // extern "C"

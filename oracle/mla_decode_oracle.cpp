// TEST INFRASTRUCTURE -- not part of the product path.
//
// FP64 oracle for paged MLA decode attention.  It is the plain definition
// (Eq. 1 of the paper, with the MLA sharing of Section 2.2: one latent row per
// key is used as K (576 columns) and its first 512 columns as V), written out
// without tiling, online softmax, or any of the paper's rescaling machinery:
//
//   s_j  = scale * sum_d q[d] * k_j[d]          for every visible key j
//   m    = max_j s_j,  l = sum_j exp(s_j - m)
//   out  = sum_j exp(s_j - m) * k_j[0:512] / l,   lse = m + ln(l)
//
// Visibility (not in the paper; decode with Sq speculative tokens): query token
// t of sequence b sees key j iff 0 <= j < N_b and j <= N_b - Sq + t.  A row with
// no visible key returns out = 0 and lse = -inf.
//
// Inputs are bf16 bit patterns widened exactly to double.  This file shares no
// code with the CUDA path and may only be used by tests, the smoke check and
// the benchmark's CPU-baseline leg.
//
// Pins (tests/test_oracle_pins.py): brute force on tiny inputs, uniform logits
// -> mean of V and lse = ln(count), a dominant key -> its V row, page
// permutation invariance, Sq=2 vs Sq=1 relations, scipy softmax/logsumexp.

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

inline double bf16_to_double(uint16_t b) {
  uint32_t u = static_cast<uint32_t>(b) << 16;
  float f;
  std::memcpy(&f, &u, sizeof(f));
  return static_cast<double>(f);
}

// One (b, t, h) row.  Returns 0 on success, 1 if a block-table entry is out of range.
int one_row(const uint16_t* q, const uint16_t* kv, const int32_t* block_table, const int32_t* seqlens,
            double scale, int Sq, int H, int num_blocks, int max_blocks_per_seq, int b, int t, int h,
            double* out, double* lse) {
  const long n_b = seqlens[b];
  long visible = n_b - Sq + t + 1;  // keys 0 .. N_b - Sq + t
  if (visible > n_b) visible = n_b;
  for (int d = 0; d < kDv; ++d) out[d] = 0.0;
  if (visible <= 0) {
    *lse = -std::numeric_limits<double>::infinity();
    return 0;
  }
  const uint16_t* qrow = q + ((static_cast<size_t>(b) * Sq + t) * H + h) * kDqk;
  double qd[kDqk];
  for (int d = 0; d < kDqk; ++d) qd[d] = bf16_to_double(qrow[d]);

  std::vector<double> s(static_cast<size_t>(visible));
  double m = -std::numeric_limits<double>::infinity();
  for (long j = 0; j < visible; ++j) {
    const long blk = j / kPage;
    if (blk >= max_blocks_per_seq) return 1;
    const int32_t page = block_table[static_cast<size_t>(b) * max_blocks_per_seq + blk];
    if (page < 0 || page >= num_blocks) return 1;
    const uint16_t* krow = kv + (static_cast<size_t>(page) * kPage + (j % kPage)) * kDqk;
    double acc = 0.0;
    for (int d = 0; d < kDqk; ++d) acc += qd[d] * bf16_to_double(krow[d]);
    s[j] = acc * scale;
    if (s[j] > m) m = s[j];
  }
  double l = 0.0;
  for (long j = 0; j < visible; ++j) {
    const double p = std::exp(s[j] - m);
    l += p;
    const int32_t page = block_table[static_cast<size_t>(b) * max_blocks_per_seq + j / kPage];
    const uint16_t* krow = kv + (static_cast<size_t>(page) * kPage + (j % kPage)) * kDqk;
    for (int d = 0; d < kDv; ++d) out[d] += p * bf16_to_double(krow[d]);
  }
  for (int d = 0; d < kDv; ++d) out[d] /= l;
  *lse = m + std::log(l);
  return 0;
}

}  // namespace

extern "C" {

// Full problem.  out: double [B, Sq, H, 512]; lse: double [B, Sq, H].
// n_threads <= 0 uses the OpenMP default.  Returns 0, or 1 on a bad block-table entry.
int oracle_mla_decode(const uint16_t* q, const uint16_t* kv, const int32_t* block_table,
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
    bad |= one_row(q, kv, block_table, seqlens, scale, Sq, H, num_blocks, max_blocks_per_seq, b, t, h,
                   out + r * kDv, lse + r);
  }
  return bad;
}

// Selected rows only.  rows: int32 [n_rows, 3] = (b, t, h); out: double [n_rows, 512]; lse: double [n_rows].
int oracle_mla_decode_rows(const uint16_t* q, const uint16_t* kv, const int32_t* block_table,
                           const int32_t* seqlens, double scale, int B, int Sq, int H, int num_blocks,
                           int max_blocks_per_seq, const int32_t* rows, int n_rows, double* out,
                           double* lse, int n_threads) {
  int bad = 0;
#ifdef _OPENMP
  if (n_threads > 0) omp_set_num_threads(n_threads);
#endif
#pragma omp parallel for schedule(dynamic, 1) reduction(| : bad)
  for (int i = 0; i < n_rows; ++i) {
    const int b = rows[3 * i], t = rows[3 * i + 1], h = rows[3 * i + 2];
    if (b < 0 || b >= B || t < 0 || t >= Sq || h < 0 || h >= H) {
      bad |= 1;
      continue;
    }
    bad |= one_row(q, kv, block_table, seqlens, scale, Sq, H, num_blocks, max_blocks_per_seq, b, t, h,
                   out + static_cast<size_t>(i) * kDv, lse + i);
  }
  return bad;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

}  // extern "C"

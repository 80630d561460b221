// Shared definitions of the libamla kernels: problem constants, the parameter block, the split-KV
// schedule arithmetic (host + device), and the per-row scalar recurrence of Algorithm 2.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace amla {

constexpr int kDqk = 576;      // K width: 512 latent + 64 RoPE columns (Section 3.1)
constexpr int kDv = 512;       // V width: the latent columns
constexpr int kPage = 64;      // keys per cache page == keys per tile
constexpr int kRowBlock = 128; // query rows per work item (= MMA M)
constexpr float kLog2e = 1.4426950408889634f;
constexpr float kLn2 = 0.6931471805599453f;

// Status word kept at workspace[0].
constexpr int kStatusOk = 0;
constexpr int kStatusTimeout = 1;

struct DecodeParams {
  const __nv_bfloat16* q;        // [B, Sq, H, 576] == [B, R, 576]
  const __nv_bfloat16* kv;       // [num_blocks, 64, 576]
  const int32_t* block_table;    // [B, max_blocks_per_seq]
  const int32_t* seqlens;        // [B]
  __nv_bfloat16* out;            // [B, R, 512]
  float* lse;                    // [B, R]
  int* status;                   // workspace status word
  const int* prefix;             // [n_items + 1] linear tile index of each item's first tile
  float* part_o;                 // normalised partial outputs of split items: [2 * P * item_rows][512] half precision, then
                                 // [2 * P * item_rows][16] scale bytes (see "Split partials" below)
  float* part_lse;               // [2 * P, 128]      partial lse (natural log)
  int2* item_info;               // [n_items] (slot of the item's first partial, number of parts it is split over), written by
                                 // the decode kernel for every item it touches, read by the combine
  float scale_log2;              // softmax_scale * log2(e)
  float tau;                     // lazy-reference threshold in octaves (0 = move the reference with every new maximum)
  float out_scale;               // factor on the normalised output (1; the dequantisation scale of an FP8 cache's V)
  int B, Sq, H;
  int R;                         // Sq * H query rows per sequence
  int nrb;                       // row blocks per sequence = ceil(R / 128)
  int n_items;                   // B * nrb
  int num_blocks, max_blocks_per_seq;
  int P;                         // parts the linear tile range is cut into
  int fused_plan;                // the decode kernel computes `prefix` itself (few items), no schedule kernel
  int flags;
  int tile_keys;                 // keys per schedule tile: 64 (one page) or 128 (two pages, the 256-row kernel)
  int item_rows;                 // query rows per work item: 128, or 256 for the 256-row kernel (nrb counts these)
  int ovh;                       // schedule positions that stand for the cost of starting an item
  unsigned long long* trace;     // timeline buffer of a -DAMLA_TRACE build, else unused (nullptr)
};

// Optional per-role timeline (compiled in with -DAMLA_TRACE only): every stamp is the SM's cycle
// counter, stored at trace[(part * kTraceEvents + event) * kTraceTiles + index].
constexpr int kTraceEvents = 32;
constexpr int kTraceTiles = 96;
#ifdef AMLA_TRACE
#define AMLA_STAMP(prm, part, ev, idx)                                                                      \
  do {                                                                                                      \
    if ((prm).trace && static_cast<unsigned>(idx) < static_cast<unsigned>(amla::kTraceTiles))                \
      (prm).trace[(static_cast<size_t>(part) * amla::kTraceEvents + (ev)) * amla::kTraceTiles + (idx)] =     \
          static_cast<unsigned long long>(clock64());                                                       \
  } while (0)
#else
#define AMLA_STAMP(prm, part, ev, idx) do { } while (0)
#endif
// Detailed stamps (several per ring slot) perturb the issuer loops; -DAMLA_TRACE=2 turns them on.
#if defined(AMLA_TRACE) && AMLA_TRACE >= 2
#define AMLA_STAMP2(prm, part, ev, idx) AMLA_STAMP(prm, part, ev, idx)
#else
#define AMLA_STAMP2(prm, part, ev, idx) do { } while (0)
#endif

// ---------------------------------------------------------------------------------------------
// Split-KV schedule.  Items (sequence b, row block rb) in order it = b * nrb + rb own
// ceil(N_b / tile_keys) tiles each (a tile is one 64-key page for the 128-row kernel, two for the 256-row one).  Starting an item costs a cluster a fixed amount of time (its Q rows,
// the pipeline fill, the epilogue) that is worth about kUnitOverheadTiles tiles, so the schedule
// balances a linear range in which every non-empty item but the first is preceded by that many
// overhead positions: prefix[it] is the position where item `it` begins (overhead first, then its tiles),
// L = prefix[n_items] the total, and part p owns positions [p*L/P, (p+1)*L/P).  A part does the
// tiles whose positions it owns; overhead positions carry no work.
// ---------------------------------------------------------------------------------------------
#ifndef AMLA_UNIT_OVERHEAD_TILES
#define AMLA_UNIT_OVERHEAD_TILES 6            // 128-row kernel: in 64-key pages (a build-time knob for tuning runs)
#endif
constexpr int kUnitOverheadTiles = AMLA_UNIT_OVERHEAD_TILES;
#ifndef AMLA_QUAD_OVERHEAD_TILES
#define AMLA_QUAD_OVERHEAD_TILES 5            // 256-row kernel: in 128-key tiles (a build-time knob for tuning runs)
#endif
constexpr int kQuadOverheadTiles = AMLA_QUAD_OVERHEAD_TILES;
constexpr int kFusedPlanMaxItems = 2048;   // up to this many items every decode CTA computes the prefix itself

// Overhead positions in front of item `it`: none for the first item, which opens the first part anyway (every
// part pays for one start; the positions stand for the additional ones).
__host__ __device__ inline int item_overhead(int it, int ovh) { return it > 0 ? ovh : 0; }
// Schedule length of an item: its tiles plus the start-up overhead (nothing for an empty sequence).
__host__ __device__ inline int schedule_length(int seqlen, int it, int tile_keys, int ovh) {
  const int n = seqlen < 0 ? 0 : seqlen;
  const int tiles = (n + tile_keys - 1) / tile_keys;
  return tiles > 0 ? tiles + item_overhead(it, ovh) : 0;
}

struct Plan {
  const int* prefix;
  int n_items;
  int L;
  int P;
  int ovh;
  bool wide;     // L * P does not fit 31 bits: the part arithmetic needs 64-bit division (slow on the device)

  // With fewer positions than parts only the first L parts exist (one position each).
  __host__ __device__ static Plan make(const int* prefix, int n_items, int max_parts, int ovh) {
    Plan pl;
    pl.prefix = prefix;
    pl.ovh = ovh;
    pl.n_items = n_items;
    pl.L = prefix[n_items];
    pl.P = pl.L < max_parts ? (pl.L > 0 ? pl.L : 1) : max_parts;
    pl.wide = static_cast<long long>(pl.L) * pl.P >= (1ll << 31);
    return pl;
  }
  // floor(a * b / c) for 0 <= a <= c-ish operands of the schedule; 32-bit unless the product could overflow
  __host__ __device__ int muldiv(int a, int b, int c) const {
    if (!wide) return static_cast<int>(static_cast<unsigned>(a) * static_cast<unsigned>(b) / static_cast<unsigned>(c));
    return static_cast<int>((static_cast<long long>(a) * b) / c);
  }
  __host__ __device__ int part_start(int p) const {
    if (p >= P) return L;
    return muldiv(p, L, P);
  }
  __host__ __device__ int part_of_tile(int g) const {
    int p = muldiv(g, P, L);
    if (p > P - 1) p = P - 1;
    while (p + 1 < P && part_start(p + 1) <= g) ++p;
    while (p > 0 && part_start(p) > g) --p;
    return p;
  }
  // Largest item index whose first tile is <= g (zero-tile items are skipped automatically).
  __host__ __device__ int item_of_tile(int g) const {
    int lo = 0, hi = n_items - 1;
    while (lo < hi) {
      int mid = (lo + hi + 1) >> 1;
      if (prefix[mid] <= g) lo = mid; else hi = mid - 1;
    }
    return lo;
  }
  // Position of the first tile of a non-empty item.
  __host__ __device__ int first_tile(int it) const { return prefix[it] + item_overhead(it, ovh); }
  // Parts [p_first, p_last] that hold tiles of item `it`; returns the split count (0 for an empty item).
  __host__ __device__ int item_parts(int it, int* p_first, int* p_last) const {
    const int e = prefix[it + 1];
    if (e <= prefix[it]) { *p_first = 0; *p_last = -1; return 0; }
    const int a = first_tile(it);
    *p_first = part_of_tile(a);
    *p_last = part_of_tile(e - 1);
    return *p_last - *p_first + 1;
  }
  // Partial slot of the unit (part p, item it): a part has at most two partial units, the one that
  // began in an earlier part / begins exactly at the part start (slot 2p) and a later one (2p+1).
  __host__ __device__ int slot_of(int p, int it, int p_first) const {
    return 2 * p + ((p == p_first && prefix[it] > part_start(p)) ? 1 : 0);
  }
  // The same from what item_info holds: slot of split s (0 = the part where the item begins) of an item
  __host__ __device__ static int slot_of_split(int first_slot, int s) { return s == 0 ? first_slot : 2 * ((first_slot >> 1) + s); }
};

// ---------------------------------------------------------------------------------------------
// Split partials.  A part that holds some of an item's tiles leaves the item's normalised output rows for the
// combine kernel.  They travel in half precision (the combine rounds its result to bf16 anyway; a half has three
// more mantissa bits), each 32-column chunk of a row scaled by a power of two so that its largest magnitude lies in
// [1, 2): the chunk's scale byte is the biased FP32 exponent of that magnitude, the stored halves are value *
// 2^(127 - byte), and value = half * 2^(byte - 127) exactly (byte 0: a chunk of zeros).  Half the bytes of FP32
// partials, whatever the range of V.
// ---------------------------------------------------------------------------------------------
__host__ __device__ inline size_t partial_rows(const DecodeParams& prm) { return static_cast<size_t>(2) * prm.P * prm.item_rows; }
__device__ __forceinline__ uint16_t* partial_halves(const DecodeParams& prm) { return reinterpret_cast<uint16_t*>(prm.part_o); }
__device__ __forceinline__ uint8_t* partial_scales(const DecodeParams& prm) {
  return reinterpret_cast<uint8_t*>(prm.part_o) + partial_rows(prm) * kDv * sizeof(uint16_t);
}
// scale byte and the factor 2^(127 - byte) for a chunk whose largest magnitude is max_abs.  The byte is the
// magnitude's exponent field kept within [64, 253]: the factor stays below 2^64, so it can be folded into another
// finite factor without overflow (chunks below 2^-63 lose precision that nothing downstream can see), and is normal.
__device__ __forceinline__ uint32_t partial_scale_byte(float max_abs, float* factor) {
  const uint32_t e = min(max((__float_as_uint(max_abs) >> 23) & 0xffu, 64u), 253u);
  *factor = __uint_as_float((254u - e) << 23);
  return e;
}
__device__ __forceinline__ float partial_unscale(uint32_t scale_byte) { return __uint_as_float(scale_byte << 23); }
__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  uint32_t r;
  asm("cvt.rn.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(hi), "f"(lo));
  return r;
}
__device__ __forceinline__ float2 unpack_f16x2(uint32_t h2) {
  float lo, hi;
  asm("{\n\t.reg .b16 a, b;\n\tmov.b32 {a, b}, %2;\n\tcvt.f32.f16 %0, a;\n\tcvt.f32.f16 %1, b;\n\t}" : "=f"(lo), "=f"(hi) : "r"(h2));
  return make_float2(lo, hi);
}

// ---------------------------------------------------------------------------------------------
// Lemma 3.1: F * 2^n == AS_FP32(AS_INT32(F) + n * 2^23) for normal F and 0 < E + n < 255.
// The guarded form adds to the magnitude bits and clamps at zero, so exact zeros stay zero and
// values that would fall below the normal range become zero/denormal instead of wrapping.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float exponent_add_guarded(float f, int n_bits) {
  const int i = __float_as_int(f);
  const int mag = max((i & 0x7fffffff) + n_bits, 0);
  return __int_as_float(mag | (i & 0x80000000));
}
__device__ __forceinline__ float exponent_add_raw(float f, int n_bits) {
  return __int_as_float(__float_as_int(f) + n_bits);
}

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float log2f_approx(float x) {
  float y;
  asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ float bf16_round(float x) {
  return __bfloat162float(__float2bfloat16_rn(x));
}

// ---------------------------------------------------------------------------------------------
// Per-row running state and the scalar part of one tile step, in the base-2 domain:
// a_j = s_j * log2(e), so exp(s_j - m) = 2^(a_j - m2) and n_i = round(-m_i / ln 2) = round(-m2).
//
// The reference m2 that P, l and O are expressed against is the running maximum of Algorithm 2 when
// tau == 0.  With tau > 0 it is moved only when a tile's maximum exceeds it by more than tau octaves
// (then to that maximum); in between P may reach 2^tau instead of 1, which bf16 P and the FP32
// accumulators hold without loss, and the accumulator needs no rescale.  Lines 6-12 of Algorithm 2
// are evaluated at the moves, with the stale reference in the place of m_{i-1}.
// ---------------------------------------------------------------------------------------------
struct RowState {
  float m2;      // reference of a_j (-inf before the first visible key)
  float l;       // running row sum of P against that reference (unscaled FP32, Algorithm 2 line 6)
  float n;       // n_i of the last move
  float c;       // c_i of the last move (Appendix A: r_i / r'_i = S16 / S32)
  float s_out;   // scale folded into P since the last move (S16, S32 or 1 depending on the mode)
};

__device__ __forceinline__ void row_state_init(RowState& st) {
  st.m2 = -INFINITY; st.l = 0.f; st.n = 0.f; st.c = 1.f; st.s_out = 1.f;
}

// Result of the scalar step for one row and one tile.
struct RowStep {
  float m2_sub;   // value to subtract inside the exponential (0 when the row has no visible key yet)
  float p_scale;  // factor folded into P before the bf16 cast
  float l_up;     // exp2(m2_old - m2_new), multiplies the old row sum (and the old O in FMUL mode)
  int n_bits;     // integer added to the accumulator's bit pattern (0 = leave the row alone)
};

// mode: 0 = Algorithm 2, 1 = exact fold (Eq. 3), 2 = FP32 multiply (Algorithm 1).
template <int kMode>
__device__ __forceinline__ RowStep row_step(RowState& st, float tile_max2, float tau) {
  RowStep r;
  const float m_old = st.m2;
  r.n_bits = 0;
  r.l_up = 1.f;
  if (!(tile_max2 > m_old + tau)) {   // reference stays (also: nothing visible in this tile)
    r.m2_sub = (m_old == -INFINITY) ? 0.f : m_old;
    r.p_scale = st.s_out;
    return r;
  }
  const float m_new = tile_max2;     // > m_old
  const bool started = m_old != -INFINITY;
  r.m2_sub = m_new;
  r.l_up = started ? ex2_approx(m_old - m_new) : 0.f;
  if (kMode == 2) {
    r.p_scale = 1.f;
    st.s_out = 1.f;
  } else {
    const float n_i = rintf(-m_new);                       // Alg. 2 line 6
    const float s32 = ex2_approx(n_i + m_new);             // line 7: 1/r_i in [1/sqrt2, sqrt2]
    const int dn = static_cast<int>(fmaxf(n_i - st.n, -30.f));   // line 11
    if (kMode == 0) {
      const float s16 = bf16_round(s32);                   // line 8
      const float c_i = __fdividef(s16, s32);              // Appendix A: c_i = r_i / r'_i
      if (started) {
        const float eps = 1.5f * (__fdividef(c_i, st.c) - 1.f);           // line 9
        r.n_bits = dn * (1 << 23) + __float2int_rn((eps + 1e-6f) * 8388608.f);   // line 12
      }
      st.c = c_i;
      r.p_scale = s16;                                     // line 10
      st.s_out = s16;
    } else {
      if (started) r.n_bits = dn * (1 << 23);              // 0 when n_i did not change
      r.p_scale = s32;
      st.s_out = s32;
    }
    st.n = n_i;
  }
  st.m2 = m_new;
  return r;
}

}  // namespace amla

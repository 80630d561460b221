// Tensor-core MLA decode kernel for sequences with more than 128 query rows (S_q >= 2 with 128 heads), sm_100a.
//
// A cluster of four CTAs works on one block of 256 query rows and a range of 128-key tiles (two cache pages):
//
//   score pair (cluster ranks 0, 1)   CTA j keeps rows 128 j .. 128 j + 127 of Q (latent part in tensor memory, RoPE
//       part in shared memory) and loads ONE page of every tile: S = Q K^T is a pair MMA (M = 256, N = 128, K = 16,
//       issued by rank 0) whose B operand is split over the two CTAs, so that every key row enters the shared
//       memory of one SM only and serves all 256 query rows.  Each CTA runs the softmax of its own 128 rows
//       (Algorithm 2's per-row recurrence, lines 5-12; two threads per row, one per page of the tile) and ships
//       P~ = bf16(P * S16) and the per-row integers N to "its" value CTA by asynchronous remote stores.
//   value pair (cluster ranks 2, 3)   CTA j holds the FP32 accumulator O of rows 128 j .. in its tensor memory; the
//       P~ V product is a pair MMA (M = 256, N = 256) whose B operand (V: 128 of the 256 columns per CTA) is again
//       split, so each value CTA loads half of every V tile.  The correction warps apply N to the bit patterns of O
//       (lines 13-16; Lemma 3.1); the epilogue divides by l * S16 (line 20).
//
// The roles, their rings and the order [QK^T(i+1), P~V(i), softmax(i+1)] (the paper's [C1, C2, V1] steady state,
// Section 4.1) are those of the 128-row kernel; what changes is that the operand traffic per SM and key is halved,
// which is what bounds that kernel.  Loads are plain TMA tile loads of each CTA into its own shared memory (no
// multicast); the bytes of both halves are counted on one barrier of the pair's even CTA.
//
// All waits are bounded; on expiry the kernel records kStatusTimeout and unwinds.
#include <atomic>
#include <type_traits>

#include "amla_common.cuh"
#include "amla_sm100.cuh"
#include "amla_epilogue.cuh"

namespace amla {

using namespace sm100;

namespace {

constexpr int kThreads = 32 * 10;   // warps 0-3 and 6-9: softmax (score CTAs) / correction + epilogue (value CTAs), 4: TMA producers, 5: MMA issuer or relay, TMEM alloc
constexpr int kTileKeys = 2 * kPage;                 // keys per schedule tile
constexpr int kItemRows = 2 * kRowBlock;             // query rows per work item
constexpr uint32_t kBoxBytes = 64 * 64 * 2;          // one 64-key x 64-column TMA box
constexpr uint32_t kPBytes = 128 * 64 * 2;           // P~ of one page: 128 rows x 128 B
constexpr uint32_t kNOff = kPBytes;                  // ... followed by the 128 per-row integers
constexpr uint32_t kFinOff = kPBytes + 128 * 4;      // ... and, with a unit's last page, 128 x (1/(l*S16), lse)
constexpr uint32_t kPXfer = kFinOff;
constexpr uint32_t kPXferLast = kFinOff + 128 * 8;
constexpr uint32_t kPStride = 18 * 1024;
constexpr int kNumP = 4;                             // P buffers in a value CTA (pages the softmax may run ahead)

// ---- score CTA
constexpr int kNumKSlots = 6;                        // two tiles in flight per CTA
constexpr uint32_t kKSlotBytes = 3 * kBoxBytes;      // 64 keys x 192 columns: [8 row groups][3 blocks][8 rows][128 B]
constexpr uint32_t kKGroupStride = 3 * 1024;
constexpr uint32_t kOffQRope = 0;                    // 128 rows x 64 bf16, 128-byte swizzle
constexpr uint32_t kOffXchg = 128 * 64 * 2;          // float [2 exchanges in flight][2 warpgroups][128 rows]: what the two threads of a row tell each other
constexpr uint32_t kOffStage = kOffXchg + 2 * 1024;  // [2][8 softmax warps] x 4 KB: a warp's 32 rows of P~ in the byte order of the P buffer, two tiles in flight
constexpr uint32_t kOffK = kOffStage + 2 * 8 * 4096;
constexpr uint32_t kEndA = kOffK + kNumKSlots * kKSlotBytes;
// ---- value CTA
constexpr int kNumVSlots = 4;
constexpr uint32_t kVHalfBytes = 2 * kBoxBytes;      // 64 keys x 128 columns: [2 blocks][64 keys][128 B]
constexpr uint32_t kVSlotBytes = 2 * kVHalfBytes;    // one page: this CTA's 128 columns of either 256-column half of V
constexpr uint32_t kOffV = 0;
constexpr uint32_t kOffP = kNumVSlots * kVSlotBytes;
constexpr uint32_t kEndB = kOffP + kNumP * kPStride;
// ---- all four: barriers at the same offset, so that one multicast commit reaches them
constexpr uint32_t kOffBars = kEndA > kEndB ? kEndA : kEndB;
constexpr uint32_t kBarBytes = 320;
#ifdef AMLA_TRACE
constexpr int kSmemPlanItems = 4;                    // trace builds: the room goes to the stamps
#else
constexpr int kSmemPlanItems = 64;
#endif
constexpr uint32_t kOffPlan = kOffBars + kBarBytes;
constexpr uint32_t kOffSeqlens = kOffPlan + ((kSmemPlanItems + 1) * 4 + 15) / 16 * 16;
#ifdef AMLA_TRACE
// trace builds: every CTA keeps its stamps (low 32 bits of its SM's cycle counter) in shared memory, so that taking
// one does not put a global store in front of the role's next release, and dumps them when it is done
constexpr int kQTraceEvents = 16, kQTraceIdx = 10;
constexpr uint32_t kOffTrace = kOffSeqlens + kSmemPlanItems * 4;
constexpr uint32_t kSmemBytes = kOffTrace + kQTraceEvents * kQTraceIdx * 4;
#define QSTAMP(smem_base_, ev, idx)                                                                          \
  do {                                                                                                       \
    if (static_cast<unsigned>(idx) < static_cast<unsigned>(kQTraceIdx))                                      \
      st_shared_b32((smem_base_) + kOffTrace + ((ev) * kQTraceIdx + (idx)) * 4, static_cast<uint32_t>(clock64())); \
  } while (0)
// event 15 holds wall-clock stamps (global timer, ns) of the kernel's phases, comparable across SMs and kernels
#define QSTAMP_NS(smem_base_, idx)                                                                           \
  do {                                                                                                       \
    if (static_cast<unsigned>(idx) < static_cast<unsigned>(kQTraceIdx))                                      \
      st_shared_b32((smem_base_) + kOffTrace + (15 * kQTraceIdx + (idx)) * 4, static_cast<uint32_t>(global_timer_ns())); \
  } while (0)
#else
constexpr uint32_t kSmemBytes = kOffSeqlens + kSmemPlanItems * 4;
#define QSTAMP(smem_base_, ev, idx) do { } while (0)
#define QSTAMP_NS(smem_base_, idx) do { } while (0)
#endif
static_assert(kSmemBytes <= 232448, "exceeds the shared memory a block can opt in to");
static_assert(kNumP == 4, "the two staging blocks per softmax warp rely on it: the P V awaited before a page is sent is that of the page four back, which used the same block");
static_assert(kOffK % 1024 == 0 && kOffP % 1024 == 0, "swizzled tiles need 1024-byte alignment");

constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kQCol = 0;            // score CTA: latent part of Q, 256 columns (two bf16 per column)
constexpr uint32_t kSCol = 256;          // score CTA: S buffers, 2 x 128 columns

constexpr uint16_t kMaskScore = 0x3, kMaskValue = 0xC, kMaskAll = 0xF;

// X_PV exists in all four CTAs: PVDONE in the value CTAs, "P buffer free" in the score CTAs.  Barriers marked (R)
// gather warps of both CTAs of a pair for the MMA issuer in the even CTA: the warps of either CTA arrive on their
// own CTA's copy (a remote arrival with cluster-scope release stalls the arriving thread for thousands of cycles),
// and in the odd CTA the otherwise idle warp 5 relays each completed phase as ONE arrival on the even CTA's copy.
enum { X_PV = 0, X_COMMON = X_PV + kNumP };
enum { A_KFULL = X_COMMON /* even CTA */, A_KEMPTY = A_KFULL + kNumKSlots, A_SFULL = A_KEMPTY + kNumKSlots, A_SEMPTY = A_SFULL + 2 /*R*/,
       A_XCHG = A_SEMPTY + 2, A_QREADY = A_XCHG + 4 /*R*/, A_QFREE, A_QFULL, A_QDONE = A_QFULL + kNumKSlots, A_NUM = A_QDONE + kNumKSlots };
enum { B_VFULL = X_COMMON /* even CTA */, B_VEMPTY = B_VFULL + kNumVSlots, B_PFULL = B_VEMPTY + kNumVSlots, B_OREADY = B_PFULL + kNumP /*R*/,
       B_NUM = B_OREADY + kNumP };
static_assert(A_NUM * 8 + 8 <= kBarBytes && B_NUM * 8 + 8 <= kBarBytes, "barrier area too small");

struct Unit {
  int b, r0, n_b, t0, t1, it;      // r0: first row of the 256-row block; t0, t1: 128-key tiles; it: item index
};

struct UnitIter {
  const DecodeParams& prm;
  Plan plan;
  int p, g, g1;
  const int* seqlens;
  __device__ UnitIter(const DecodeParams& prm_, const int* prefix, const int* seqlens_, int part)
      : prm(prm_), plan(Plan::make(prefix, prm_.n_items, prm_.P, prm_.ovh)), p(part), seqlens(seqlens_) {
    if (plan.L <= 0 || p >= plan.P) { g = g1 = 0; }
    else { g = plan.part_start(p); g1 = plan.part_start(p + 1); }
  }
  __device__ bool next(Unit& u) {
    int it, a;
    while (true) {
      if (g >= g1) return false;
      it = plan.item_of_tile(g);
      a = plan.first_tile(it);
      const int e = plan.prefix[it + 1];
      const int lo = max(g, a), hi = min(e, g1);
      g = min(e, g1);
      if (hi > lo) { u.t0 = lo - a; u.t1 = hi - a; break; }
    }
    u.it = it;
    u.b = it / prm.nrb;
    u.r0 = (it % prm.nrb) * kItemRows;
    u.n_b = min(max(seqlens[u.b], 0), prm.max_blocks_per_seq * kPage);
    return true;
  }
  // Partial slot of the unit, -1 if its item lies in one part (several divisions: only the epilogue asks);
  // *info = what the combine needs to know about the item
  __device__ int slot_of(const Unit& u, int2* info) const {
    int p_first, p_last;
    const int nsplit = plan.item_parts(u.it, &p_first, &p_last);
    *info = make_int2(plan.slot_of(p_first, u.it, p_first), nsplit);
    return nsplit == 1 ? -1 : plan.slot_of(p, u.it, p_first);
  }
};

// Finds the unit that holds the k-th tile of this cluster's part; k never decreases between calls.
struct Cursor {
  UnitIter it;
  Unit u;
  int base;
  int ord;       // ordinal of the current unit within the part
  bool valid;
  __device__ Cursor(const DecodeParams& prm, const int* prefix, const int* seqlens, int part) : it(prm, prefix, seqlens, part), base(0), ord(0) { valid = it.next(u); }
  __device__ bool locate(int k, int& local) {
    while (valid && k >= base + (u.t1 - u.t0)) { base += u.t1 - u.t0; valid = it.next(u); ++ord; }
    local = k - base;
    return valid;
  }
};

__device__ __forceinline__ void report_timeout(int* status) { atomicExch(status, kStatusTimeout); }

template <bool kClusterAcquire = false>
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
  return __all_sync(0xffffffffu, mbar_wait<kClusterAcquire>(bar, parity));
}

// One arrival per warp on a barrier of this CTA, after every lane's preceding work.
__device__ __forceinline__ void warp_arrive(uint32_t bar, int lane) {
  __syncwarp();
  if (lane == 0) mbar_arrive(bar);
}

__device__ __forceinline__ void prefetch_q_row(const DecodeParams& prm, const Unit& u, int row) {
  if (u.r0 + row < prm.R) {
    const char* p = reinterpret_cast<const char*>(prm.q + (static_cast<size_t>(u.b) * prm.R + u.r0 + row) * kDqk);
#pragma unroll
    for (int i = 0; i < 9; ++i) prefetch_l2(p + 128 * i);
  }
}

// Q comes on chip through the K ring.  At the start of a unit every ring slot of a score CTA takes a piece of the
// CTA's 128 Q rows as TMA boxes of 64 rows x one 64-column block ([row][128 B], 128-byte swizzle): slot s holds block
// s (two boxes); the eight blocks of the latent part are two more than there are slots, so the four half-blocks of
// blocks 6 and 7 ride in the spare third of slots 0-3; the RoPE block goes straight to its operand tile, counted on
// slot 0's barrier.  The eight softmax warps then move the latent blocks into tensor memory, thread = row.
constexpr uint32_t kQHalfBytes = 64 * 128;              // one box
__device__ __forceinline__ void issue_q_piece(const CUtensorMap* q_map, uint32_t smem_base, uint32_t bars, int s, int row0) {
  const uint32_t full = bars + 8u * (A_QFULL + s), dst = smem_base + kOffK + s * kKSlotBytes;
  mbar_arrive_expect_tx(full, (s == 0 ? 5 : s < 4 ? 3 : 2) * kQHalfBytes);
  tma_load_3d(dst, q_map, 0, row0, s, full);
  tma_load_3d(dst + kQHalfBytes, q_map, 0, row0 + 64, s, full);
  if (s < 4) tma_load_3d(dst + 2 * kQHalfBytes, q_map, 0, row0 + 64 * (s & 1), 6 + (s >> 1), full);
  if (s == 0) {
    tma_load_3d(smem_base + kOffQRope, q_map, 0, row0, 8, full);
    tma_load_3d(smem_base + kOffQRope + kQHalfBytes, q_map, 0, row0 + 64, 8, full);
  }
}
// 128 bytes of one row of a box (or of two stacked boxes) -> 32 tensor-memory columns (two bf16 per column)
__device__ __forceinline__ void move_q_block(uint32_t box, int row, bool valid, uint32_t taddr) {
  uint32_t x[32];
#pragma unroll
  for (int c = 0; c < 8; ++c)
    asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(x[4 * c]), "=r"(x[4 * c + 1]), "=r"(x[4 * c + 2]), "=r"(x[4 * c + 3])
                 : "r"(box + sw128_offset(row, c)));
  if (!valid) {
#pragma unroll
    for (int i = 0; i < 32; ++i) x[i] = 0;
  }
  tmem_st_32x32b_x32(taddr, x);
}

struct RoleCtx {
  uint32_t smem_base, bars, tbase;
  uint32_t peer_base, peer_bars;                // this score CTA's value CTA (cluster addresses)
  int half, tid;                                // half: which 128 rows of the 256-row block this CTA owns
  int part;
};

// One softmax warp's work on one unit.  Two threads share a query row: the thread of warpgroup A (warps 0-3) takes
// the first 64-key page of every 128-key score tile, the thread of warpgroup B (warps 6-9, which reach the same
// tensor-memory lanes as warps 2, 3, 0, 1) the second.  Each reads its 64 scores into registers (the score tile is
// free for the next QK^T from then on), the two exchange their maxima through shared memory and run Algorithm 2's
// per-row recurrence (lines 5-12) on the same inputs, so both hold the same state; the row sum of line 6 is kept as
// two partial sums that meet at the end of the unit.  P~ = bf16(P * S16) and the row's integer N (first page only:
// the second page leaves O alone) go straight into a P buffer of this CTA's value CTA by asynchronous remote stores
// counted on its barrier; with the unit's last page travel the final scalars 1/(l*S16) and lse (line 20).
// Returns (score tiles so far) << 1 | ok.
template <int kMode>
__device__ __noinline__ uint32_t softmax_unit(const DecodeParams prm, const RoleCtx c, const Unit u, uint32_t gs, uint32_t un) {
  const int tid = c.tid, wid = tid >> 5, lane = tid & 31;
  const uint32_t smem_base = c.smem_base, bars = c.bars, tbase = c.tbase;
  auto bar = [&](int i) { return bars + 8u * i; };
  bool ok = true;
  const int hsel = wid >= 6 ? 1 : 0;                   // which page of every tile
  const int quarter = wid & 3;                         // tensor-memory lane quarter of this warp
  const int r = quarter * 32 + lane;                   // query row within this CTA's 128
  const uint32_t lane_base = static_cast<uint32_t>(quarter * 32) << 16;
  const bool scale_nonneg = prm.scale_log2 >= 0.f;
  const uint32_t mask_fill = __float_as_uint(scale_nonneg ? -INFINITY : INFINITY);
  RowState st;
  row_state_init(st);
  const int tok = (u.r0 + c.half * kRowBlock + r) / prm.H;
  const int visible = min(u.n_b, u.n_b - prm.Sq + tok + 1);               // keys 0..visible-1 are seen by this row
  const int first_masked_tile = max(u.n_b - prm.Sq + 1, 0) / kTileKeys;   // tiles from here on may hold hidden keys
  uint32_t xc = gs + un;                                // exchanges so far: one per tile, one at the end of a unit
  const uint32_t xbar = bar(A_XCHG + quarter);
  // tells the row's other thread `mine`, returns what it told
  auto exchange = [&](float mine) -> float {
    const uint32_t slot = smem_base + kOffXchg + (xc & 1) * 1024;
    st_shared_b32(slot + (hsel * 128 + r) * 4, __float_as_uint(mine));
    warp_arrive(xbar, lane);
    ok = warp_wait(xbar, xc & 1);
    ++xc;
    return __uint_as_float(ld_shared_b32(slot + ((hsel ^ 1) * 128 + r) * 4));
  };

  for (int t = u.t0; t < u.t1 && ok; ++t, ++gs) {
    const uint32_t sb = gs & 1;
    ok = warp_wait(bar(A_SFULL + sb), (gs >> 1) & 1);
    if (!ok) break;
    tc_fence_after_sync();
    if (tid == 0) QSTAMP(c.smem_base, 2, gs);
    if (tid == 0 && gs == 0) QSTAMP_NS(c.smem_base, 6);
    const uint32_t scol = tbase + lane_base + kSCol + 128 * sb + 64 * hsel;
    const int nvis = visible - t * kTileKeys - 64 * hsel;    // keys of this page the row sees (may be <= 0)
    const bool last_tile = t + 1 == u.t1;
    uint32_t b0[32], b1[32];
    tmem_ld_32x32b_x32(scol, b0);
    tmem_ld_32x32b_x32(scol + 32, b1);
    tmem_wait_ld();
    tc_fence_before_sync();
    warp_arrive(bar(A_SEMPTY + sb), lane);                   // the scores are in registers
    if (tid == 0) QSTAMP(c.smem_base, 3, gs);
    auto tile_body = [&](auto general_c) {
      constexpr bool kGeneral = decltype(general_c)::value;
      constexpr bool masked = kGeneral;
      const bool scale_nn = kGeneral ? scale_nonneg : true;
      // lines 5-6: running max on the raw scores (the scale is folded into the FMA below)
      float ext = scale_nn ? -INFINITY : INFINITY, ext_b = ext;
      auto chunk_max = [&](uint32_t (&v)[32], int col0) {
        if (masked) {
#pragma unroll
          for (int i = 0; i < 32; ++i) v[i] = (col0 + i < nvis) ? v[i] : mask_fill;
        }
        if (scale_nn) {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            ext = fmax3(ext, __uint_as_float(v[i]), __uint_as_float(v[i + 1]));
            ext_b = fmax3(ext_b, __uint_as_float(v[i + 2]), __uint_as_float(v[i + 3]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            ext = fminf(ext, fminf(__uint_as_float(v[i]), __uint_as_float(v[i + 1])));
            ext_b = fminf(ext_b, fminf(__uint_as_float(v[i + 2]), __uint_as_float(v[i + 3])));
          }
        }
      };
      chunk_max(b0, 0);
      chunk_max(b1, 32);
      ext = scale_nn ? fmaxf(ext, ext_b) : fminf(ext, ext_b);
      const float mine = (nvis > 0) ? ext * prm.scale_log2 : -INFINITY;
      const float tmax = fmaxf(mine, exchange(mine));
      if (!ok) return;
      // Lazy reference: a row must move when its maximum exceeds the reference by more than tau.  The correction warp
      // that serves these 32 rows pays for a rescale as soon as one of them moves, so when one must, every row of the
      // warp whose maximum rose moves with it (moving early is always allowed: tau = 0 moves at every rise); the rows
      // then tend to stay in step and the warp rescales on far fewer tiles.
      const bool must = tmax > st.m2 + prm.tau;
      const RowStep sp = row_step<kMode>(st, tmax, __any_sync(0xffffffffu, must) ? 0.f : prm.tau);
      if (tid == 0) QSTAMP(c.smem_base, 13, gs);
      // Line 10's factor S16 goes into the exponential's argument (the remark after Algorithm 2).  The row sum of
      // line 6 is the sum of the same FP32 values, taken before the bf16 cast and divided by S16 once per tile.
      const float nsub = log2f_approx(sp.p_scale) - sp.m2_sub;
      float rs0 = 0.f, rs1 = 0.f;
      const uint64_t sc2 = pack_f32x2(prm.scale_log2, prm.scale_log2), ns2 = pack_f32x2(nsub, nsub);
      uint64_t rsa = pack_f32x2(0.f, 0.f), rsb = rsa;
      uint32_t pk[32];
      auto chunk_exp = [&](const uint32_t (&v)[32], int col0, int k0) {
        if (masked) {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float p0 = ex2_approx(fmaf(__uint_as_float(v[2 * i]), prm.scale_log2, nsub));
            float p1 = ex2_approx(fmaf(__uint_as_float(v[2 * i + 1]), prm.scale_log2, nsub));
            p0 = (col0 + 2 * i < nvis) ? p0 : 0.f;
            p1 = (col0 + 2 * i + 1 < nvis) ? p1 : 0.f;
            rs0 += p0; rs1 += p1;
            pk[k0 + i] = pack_bf16x2(p0, p1);
          }
        } else {
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            float x0, x1;
            unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1])), sc2, ns2), x0, x1);
            const float q0 = ex2_approx(x0), q1 = ex2_approx(x1);
            const uint64_t pp = pack_f32x2(q0, q1);
            if (i & 1) rsb = add_f32x2(rsb, pp); else rsa = add_f32x2(rsa, pp);
            pk[k0 + i] = pack_bf16x2(q0, q1);
          }
        }
      };
      chunk_exp(b0, 0, 0);
      chunk_exp(b1, 32, 16);
      {
        float s0, s1;
        unpack_f32x2(add_f32x2(rsa, rsb), s0, s1);
        st.l = st.l * sp.l_up + __fdividef((rs0 + s0) + (rs1 + s1), sp.p_scale);   // this thread's share of the row sum
      }
      // ---- ship the page: P~ (128 B of this row), the row's word N, and with the unit's last page the final scalars.
      // The warp's 32 rows are a contiguous 4 KB block of the P buffer: they are staged in a block of the warp's own
      // and moved by the copy engine (remote stores by the threads would hold the warp at the rate of the SM-to-SM
      // link, ~900 clk per tile).  Two staging blocks alternate; the one written now was last read for the page four
      // pages back in the same P buffer, whose P V -- awaited next -- cannot have run before that copy had landed.
      const uint32_t gp = 2 * gs + hsel;                     // page number within the cluster's work
      const uint32_t pb = gp % kNumP;
      ok = warp_wait(bar(X_PV + pb), ((gp / kNumP) & 1) ^ 1);     // the P V that last read the buffer is done
      if (!ok) return;
      const uint32_t stage = smem_base + kOffStage + ((gs & 1) * 8 + hsel * 4 + quarter) * 4096;
#pragma unroll
      for (int cc = 0; cc < 8; ++cc)
        st_shared_v4(stage + sw128_offset(lane, cc), pk[4 * cc], pk[4 * cc + 1], pk[4 * cc + 2], pk[4 * cc + 3]);
      fence_proxy_async_smem();
      __syncwarp();
      const bool with_fin = last_tile && hsel == 1;
      const uint32_t pfull = c.peer_bars + 8u * (B_PFULL + pb);
      const uint32_t dstp = c.peer_base + kOffP + pb * kPStride;
      if (quarter == 0 && lane == 0) { QSTAMP(c.smem_base, 5, gp); mbar_arrive_expect_tx_cluster(pfull, with_fin ? kPXferLast : kPXfer); }
      if (lane == 0) bulk_copy_to_cluster(dstp + quarter * 4096, stage, 4096, pfull);
      const uint32_t nword = (kMode == 2) ? __float_as_uint(hsel == 0 ? sp.l_up : 1.f)
                                          : static_cast<uint32_t>(hsel == 0 ? sp.n_bits : 0);
      st_async_b32(dstp + kNOff + r * 4, nword, pfull);
      if (tid == 0) QSTAMP(c.smem_base, 4, gp);
      if (last_tile) {
        // line 20 scalars: 1 / (l * S16) and lse = m + ln l, from both threads' shares of the row sum
        const float l_all = st.l + exchange(st.l);
        if (ok && hsel == 1) {
          const bool live = l_all > 0.f;
          const float inv = live ? prm.out_scale / (l_all * st.s_out) : 0.f;
          const float lse = live ? (st.m2 + log2f(l_all)) * kLn2 : -INFINITY;
          st_async_v2(dstp + kFinOff + r * 8, __float_as_uint(inv), __float_as_uint(lse), pfull);
        }
      }
    };
    if (t >= first_masked_tile || !scale_nonneg) tile_body(std::true_type{});
    else tile_body(std::false_type{});
  }
  return (gs << 1) | (ok ? 1u : 0u);
}

// Relay warp of a pair's odd CTA: lane l < n_lanes watches barrier `first + l` of this CTA and passes each of its
// `phases` completed phases on as one arrival on the same barrier of the even CTA.  The lanes poll without blocking
// and in lockstep (a blocking wait in one lane of a diverged warp holds the other lanes back for its whole
// suspension time).  Returns false if a phase did not come within the wait limit.
template <bool kProxyFence>
__device__ __forceinline__ bool relay_phases(uint32_t bars, uint32_t lead_bars, int first, int lane, int phases) {
  const uint32_t lb = bars + 8u * (first + lane), rb = lead_bars + 8u * (first + lane);
  int k = 0;
  uint64_t t_start = global_timer_ns();
  for (uint32_t spin = 0;; ++spin) {
    bool progress = false;
    if (k < phases && mbar_probe(lb, k & 1)) {
      if (kProxyFence) fence_proxy_async_smem();
      mbar_arrive_cluster_relaxed(rb);
      ++k;
      progress = true;
    }
    if (__all_sync(0xffffffffu, k >= phases)) return true;
    if (__any_sync(0xffffffffu, progress)) t_start = global_timer_ns(); else __nanosleep(32);
    if ((spin & 1023u) == 1023u && __any_sync(0xffffffffu, global_timer_ns() - t_start > kWaitLimitNs)) return false;
  }
}

}  // namespace

template <int kMode, bool kGuard>
__global__ void __cluster_dims__(4, 1, 1) __launch_bounds__(kThreads, 1)
decode_quad_kernel(const __grid_constant__ CUtensorMap k_map, const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap q_map,
                   const DecodeParams prm) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const bool is_score = rank < 2;
  const int half = rank & 1;                 // which 128 rows of the block; the even CTA of a pair issues its MMAs
  const bool leader = half == 0;
  const int part = blockIdx.x >> 2;
  if (smem_base & 1023u) {
    if (tid == 0) report_timeout(prm.status);
    return;
  }

#ifdef AMLA_TRACE
  const uint32_t t_entry = static_cast<uint32_t>(global_timer_ns());
  for (int i = tid; i < kQTraceEvents * kQTraceIdx; i += kThreads) st_shared_b32(smem_base + kOffTrace + 4 * i, 0u);
  __syncthreads();
  if (tid == 0) st_shared_b32(smem_base + kOffTrace + (15 * kQTraceIdx + 0) * 4, t_entry);
#endif
  const uint32_t bars = smem_base + kOffBars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const uint32_t tmem_slot = bars + kBarBytes - 8;
  const uint32_t lead_bars = map_to_cta(bars, rank & ~1u);              // barrier area of this pair's even CTA
  const uint32_t myV_base = map_to_cta(smem_base, 2 + half);           // score CTA j -> value CTA j
  const uint32_t myV_bars = map_to_cta(bars, 2 + half);

  // The lengths of the first 32 items are requested before anything else, so that their latency runs under the set-up
  // below (they are inputs of the call: no kernel that this one may overlap with writes them).
  int early_len = 0;
  if (wid == 6 && prm.fused_plan && lane < prm.n_items) early_len = prm.seqlens[lane / prm.nrb];
  if (tid == 0) {
    for (int i = 0; i < kNumP; ++i) mbar_init(bar(X_PV + i), 1);
    if (is_score) {
      for (int i = 0; i < kNumKSlots; ++i) { mbar_init(bar(A_KFULL + i), 1); mbar_init(bar(A_KEMPTY + i), 1); }
      for (int i = 0; i < 2; ++i) {
        mbar_init(bar(A_SFULL + i), 1); mbar_init(bar(A_SEMPTY + i), leader ? 9 : 8);   // 8 softmax warps (+ the odd CTA's relay)
      }
      for (int i = 0; i < 4; ++i) mbar_init(bar(A_XCHG + i), 2);                        // the two warps that share 32 rows
      mbar_init(bar(A_QREADY), leader ? 9 : 8);                                         // 8 loading warps (+ relay)
      mbar_init(bar(A_QFREE), 1);
      for (int i = 0; i < kNumKSlots; ++i) {
        mbar_init(bar(A_QFULL + i), 1);
        mbar_init(bar(A_QDONE + i), (i == 1 || i == 2) ? 6 : 4);     // the warps that read a piece of Q from slot i
      }
    } else {
      for (int i = 0; i < kNumVSlots; ++i) { mbar_init(bar(B_VFULL + i), 1); mbar_init(bar(B_VEMPTY + i), 1); }
      for (int i = 0; i < kNumP; ++i) { mbar_init(bar(B_PFULL + i), 1); mbar_init(bar(B_OREADY + i), leader ? 9 : 8); }   // 8 correction warps (+ relay)
    }
    fence_mbar_init();
    prefetch_tensormap(&k_map);
    prefetch_tensormap(&v_map);
    prefetch_tensormap(&q_map);
  }
  if (wid == 5) { tmem_alloc_pair(tmem_slot, kTmemCols); tmem_relinquish_pair(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();
  tc_fence_after_sync();
  const uint32_t tbase = ld_shared_b32(tmem_slot);

  if (tid == 0) QSTAMP_NS(smem_base, 1);
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  if (tid == 0) QSTAMP_NS(smem_base, 2);
  const int* prefix = prm.prefix;
  const int* seqlens = prm.seqlens;
  if (prm.fused_plan) {
    int* ps = prm.n_items <= kSmemPlanItems ? reinterpret_cast<int*>(smem_raw + kOffPlan) : nullptr;
    if (wid == 6) {
      int* pw = const_cast<int*>(prm.prefix);
      int carry = 0;
      for (int base = 0; base < prm.n_items; base += 32) {
        const int it = base + lane;
        const int n_seq = it >= prm.n_items ? 0 : base == 0 ? early_len : prm.seqlens[it / prm.nrb];
        if (ps && it < prm.n_items) reinterpret_cast<int*>(smem_raw + kOffSeqlens)[it / prm.nrb] = n_seq;
        const int v = it < prm.n_items ? schedule_length(n_seq, it, prm.tile_keys, prm.ovh) : 0;
        int x = v;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, x, o);
          if (lane >= o) x += y;
        }
        if (it < prm.n_items) {
          pw[it] = carry + x - v;
          if (ps) ps[it] = carry + x - v;
        }
        carry += __shfl_sync(0xffffffffu, x, 31);
      }
      if (lane == 0) {
        pw[prm.n_items] = carry;
        if (ps) ps[prm.n_items] = carry;
        if (blockIdx.x == 0) *prm.status = kStatusOk;
      }
      __threadfence_block();
    }
    __syncthreads();
    if (ps) { prefix = ps; seqlens = reinterpret_cast<const int*>(smem_raw + kOffSeqlens); }
  }
  if (is_score && tid < kNumKSlots) {   // the first unit's Q is requested before the roles start: one piece per lane
    UnitIter first(prm, prefix, seqlens, part);
    Unit fu;
    if (first.next(fu)) issue_q_piece(&q_map, smem_base, bars, tid, fu.b * prm.R + fu.r0 + half * kRowBlock);
  }

  bool ok = true;
  UnitIter iter(prm, prefix, seqlens, part);
  Unit u;
  uint32_t gt = 0;      // 64-key pages processed by this cluster so far (two per tile; all roles count identically)
  uint32_t un = 0;      // units processed so far

  if (is_score) {
    // ======================================================================= score CTAs
    uint32_t gs = 0;    // score tiles so far
    if (wid < 4 || wid >= 6) {
      // ---- softmax warps: A = warps 0-3 (first page of every tile), B = warps 6-9 (second page).  At the start of
      // a unit they bring in its Q rows: A the first 256 latent columns, B the other 256 and the RoPE columns.
      const bool grp_b = wid >= 6;
      const int qr = (wid & 3) * 32 + lane;
      const uint32_t q_lane_base = static_cast<uint32_t>((wid & 3) * 32) << 16;
      const RoleCtx ctx{smem_base, bars, tbase, myV_base, myV_bars, half, tid, part};
      while (ok && iter.next(u)) {
        ok = warp_wait(bar(A_QFREE), (un & 1) ^ 1);      // the previous unit's QK^T is finished with Q
        if (!ok) break;
        tc_fence_after_sync();
        if (tid == 0) { if (un < 1) QSTAMP_NS(smem_base, 8 + 4 * un); };
        {
          // Group A moves blocks 0, 2, 4 (slots 0, 2, 4) and block 6, whose halves sit in slots 0 and 1; group B blocks
          // 1, 3, 5 and block 7 (halves in slots 2 and 3).  A warp hands a slot back after its last read from it.
          const bool valid = u.r0 + half * kRowBlock + qr < prm.R;
          const int quarter = wid & 3;
          const uint32_t kbase = smem_base + kOffK, trow = tbase + q_lane_base + kQCol, qpar = un & 1;
          const uint32_t extra_col = 32 * (grp_b ? 7 : 6);
#pragma unroll 1
          for (int i = 0; i < 3 && ok; ++i) {
            const int sl = 2 * i + (grp_b ? 1 : 0);
            ok = warp_wait(bar(A_QFULL + sl), qpar);
            if (!ok) break;
            move_q_block(kbase + sl * kKSlotBytes, qr, valid, trow + 32 * sl);
            if (grp_b ? (sl == 3 && quarter >= 2) : (sl == 0 && quarter < 2))
              move_q_block(kbase + sl * kKSlotBytes + 2 * kQHalfBytes, qr & 63, valid, trow + extra_col);
            warp_arrive(bar(A_QDONE + sl), lane);
          }
          if (!ok) break;
          if (grp_b ? (quarter < 2) : (quarter >= 2)) {     // the half-block that rides in a slot of the other group
            const int sl = grp_b ? 2 : 1;
            ok = warp_wait(bar(A_QFULL + sl), qpar);
            if (!ok) break;
            move_q_block(kbase + sl * kKSlotBytes + 2 * kQHalfBytes, qr & 63, valid, trow + extra_col);
            warp_arrive(bar(A_QDONE + sl), lane);
          }
          tmem_wait_st();
        }
        tc_fence_before_sync();
        warp_arrive(bar(A_QREADY), lane);
        if (tid == 0) { if (un < 1) QSTAMP_NS(smem_base, 9 + 4 * un); };
        if (grp_b) {                               // the next unit's Q goes to L2 while this one is computed
          UnitIter peek = iter;
          Unit nu;
          if (peek.next(nu)) prefetch_q_row(prm, nu, half * kRowBlock + qr);
        }
        const uint32_t ret = softmax_unit<kMode>(prm, ctx, u, gs, un);
        gs = ret >> 1;
        ok = (ret & 1u) != 0;
        ++un;
      }
      if (!ok && lane == 0) report_timeout(prm.status);
    } else if (wid == 4) {
      // ---- TMA producers: K.  This CTA loads page (2 t + half) of every tile t, three slots of 192 columns; lane l
      // owns ring slot l and polls without blocking.  The bytes of both CTAs' halves are counted on the even CTA's
      // "full" barrier.  A sequence's last tile may have one page only: the odd CTA then loads the first page
      // again (finite values that the softmax masks as keys beyond the sequence).
      // At the start of every unit the slot first carries the lane's piece of that unit's Q (see issue_q_piece; lane 0
      // waits for the previous unit's MMAs to let go of the RoPE tile); the first unit's pieces were requested before
      // the roles split.
      Cursor cur(prm, prefix, seqlens, part);
      bool fin = lane >= kNumKSlots;
      const bool first_out = !fin && cur.valid;
      UnitIter qit = cur.it;                  // walks the units whose Q this lane has not requested (it stands behind the first)
      Unit qu;
      bool q_left = false, q_stale = first_out;
      auto q_due = [&]() { if (q_stale) { q_left = qit.next(qu); q_stale = false; } return q_left; };
      int q_ord = first_out ? 1 : 0;          // ordinal of the unit qu
      int nq = first_out ? 1 : 0;             // pieces of Q requested for this slot
      int my_tile = lane / 3;                 // kNumKSlots = 6: lane l always loads column group l % 3, every second tile
      const int g = lane % 3;
      uint32_t par = 1;
      int k_state = 0, k_ord = 0, pending = 0;   // K slot: 0 not looked up, 1 page number at hand, 2 none left; pending: 1 Q, 2 K
      int page_id = 0;
      int issued = 0;
      const uint32_t my_full = bar(A_KFULL + lane), my_empty = bar(A_KEMPTY + lane), my_qdone = bar(A_QDONE + lane);
      const uint32_t lead_full = lead_bars + 8u * (A_KFULL + lane);
      const uint32_t dst = smem_base + kOffK + lane * kKSlotBytes;
      uint64_t t_start = global_timer_ns();
      bool progress = false;
      for (uint32_t spin = 0;; ++spin) {
        if (!fin && pending == 0) {
          if (k_state == 0) {
            int lt;
            if (cur.locate(my_tile, lt)) {
              const int t = cur.u.t0 + lt;
              const int npg = (cur.u.n_b + kPage - 1) / kPage;
              const int pg = (2 * t + half < npg) ? 2 * t + half : 2 * t;
              page_id = __ldg(prm.block_table + static_cast<size_t>(cur.u.b) * prm.max_blocks_per_seq + pg);
              k_ord = cur.ord;
              k_state = 1;
            } else {
              k_state = 2;
            }
          }
          if ((k_state == 2 || q_ord <= k_ord) && q_due()) pending = 1;
          else if (k_state == 1) pending = 2;
          else fin = true;
        }
        if (pending != 0) {
          // the slot is free when its last K load has been used up by the MMAs and its last piece of Q has been moved
          bool free_now = mbar_probe(my_empty, par) && (nq == 0 || mbar_probe(my_qdone, (nq - 1) & 1));
          if (free_now && pending == 1 && lane == 0 && q_ord > 0) free_now = mbar_probe(bar(A_QFREE), (q_ord - 1) & 1);
          if (free_now) {
            if (pending == 1) {
              issue_q_piece(&q_map, smem_base, bars, lane, qu.b * prm.R + qu.r0 + half * kRowBlock);
              q_stale = true;
              ++q_ord; ++nq;
            } else {
              if (leader) mbar_arrive_expect_tx(my_full, 2 * kKSlotBytes);
              tma_load_4d_pair(dst, &k_map, 0, 0, 3 * g, page_id * 8, lead_full);
              my_tile += 2;
              par ^= 1;
              ++issued;
              k_state = 0;
            }
            pending = 0;
            progress = true;
          }
        }
        if (__all_sync(0xffffffffu, fin)) break;
        const bool any_progress = __any_sync(0xffffffffu, progress);
        if (any_progress) t_start = global_timer_ns(); else __nanosleep(100);
        progress = false;
        if ((spin & 1023u) == 1023u && __any_sync(0xffffffffu, global_timer_ns() - t_start > kWaitLimitNs)) { ok = false; break; }
      }
      if (!ok) {
        if (lane == 0) report_timeout(prm.status);
        if (leader && issued > 0 && lane < kNumKSlots) mbar_wait(my_full, (issued - 1) & 1);   // let copies in flight land
        if (nq > 0 && lane < kNumKSlots) mbar_wait(bar(A_QFULL + lane), (nq - 1) & 1);
      }
    } else if (wid == 5) {
      // ---- MMA issuer (even CTA only): S[sb] = Q K^T for both CTAs' rows, 36 steps of K = 16 over three slots
      if (leader && lane == 0) {
        constexpr uint32_t idesc = make_idesc_bf16(256, 128, false, false);
        constexpr uint32_t dhi = smem_desc_hi_sw128(kKGroupStride);
        constexpr uint32_t qhi = smem_desc_hi_sw128(1024);
        const uint32_t klo0 = smem_desc_lo(smem_base + kOffK, 16);
        const uint32_t qlo0 = smem_desc_lo(smem_base + kOffQRope, 16);
        uint32_t slot = 0, kpar = 0;
        while (ok && iter.next(u)) {
          ok = mbar_wait<true>(bar(A_QREADY), un & 1);
          if (!ok) break;
          tc_fence_after_sync();
          for (int t = u.t0; t < u.t1 && ok; ++t, ++gs) {
            const uint32_t sb = gs & 1;
            ok = mbar_wait(bar(A_SEMPTY + sb), ((gs >> 1) & 1) ^ 1);
            if (!ok) break;
            tc_fence_after_sync();
            QSTAMP(smem_base, 0, gs);
            const uint32_t d = tbase + kSCol + 128 * sb;
            // the three slots of the tile are probed together (their latencies overlap); the blocking wait runs
            // only for one that is not there yet
            bool have[3];
            {
              uint32_t s2 = slot, p2 = kpar;
#pragma unroll
              for (int gg = 0; gg < 3; ++gg) {
                have[gg] = mbar_probe(bar(A_KFULL) + 8 * s2, p2);
                if (++s2 == kNumKSlots) { s2 = 0; p2 ^= 1; }
              }
            }
#pragma unroll
            for (int gg = 0; gg < 3; ++gg) {
              ok = ok && (have[gg] || mbar_wait(bar(A_KFULL) + 8 * slot, kpar));
              if (ok) {
                if (gg == 0) QSTAMP(smem_base, 12, gs);
                const uint32_t klo = klo0 + slot * (kKSlotBytes >> 4);
#pragma unroll
                for (int cl = 0; cl < 3; ++cl) {
                  const int cb = 3 * gg + cl;
#pragma unroll
                  for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t bd = smem_desc_join(klo + 64 * cl + 2 * kk, dhi);
                    if (cb < 8) mma_ts_pair(d, tbase + kQCol + 32 * cb + 8 * kk, bd, idesc, (cb | kk) != 0 ? 1u : 0u);
                    else mma_ss_pair(d, smem_desc_join(qlo0 + 2 * kk, qhi), bd, idesc, 1u);   // RoPE columns: Q from shared memory
                  }
                }
                mma_commit_pair_multicast(bar(A_KEMPTY) + 8 * slot, kMaskScore);
              }
              if (++slot == kNumKSlots) { slot = 0; kpar ^= 1; }
            }
            if (!ok) break;
            mma_commit_pair_multicast(bar(A_SFULL + sb), kMaskScore);
            QSTAMP(smem_base, 1, gs);
          }
          if (!ok) break;
          mma_commit_pair_multicast(bar(A_QFREE), kMaskScore);
          ++un;
        }
        if (!ok) report_timeout(prm.status);
      } else if (!leader) {
        // ---- relay (odd CTA): lanes 0, 1 pass on the completed phases of SEMPTY[lane] (the tiles with that buffer),
        // lane 2 those of QREADY (one per unit)

        int n_units = 0, n_tiles = 0;
        while (iter.next(u)) { ++n_units; n_tiles += u.t1 - u.t0; }
        const int phases = lane == 2 ? n_units : lane < 2 ? (n_tiles + 1 - lane) / 2 : 0;
        const int first = lane == 2 ? A_QREADY - 2 : A_SEMPTY;     // lane 2 lands on QREADY
        if (!relay_phases<false>(bars, lead_bars, first, lane, phases) && lane == 0) report_timeout(prm.status);
      }
    }
  } else {
    // ======================================================================= value CTAs
    if (wid < 4 || (wid >= 6 && wid < 10)) {
      // ---- correction + epilogue: thread = query row.  Warps 6-9 are the partners of warps 2, 3, 0, 1 (same
      // tensor-memory lanes): each of a pair takes one half of the row's 512 columns, in the rescale and in the epilogue.
      const bool partner = wid >= 4;
      const int r = (wid & 3) * 32 + lane;
      const uint32_t lane_base = static_cast<uint32_t>((wid & 3) * 32) << 16;
      const int c_first = partner ? 8 : 0;
      while (ok && iter.next(u)) {
        const int npages = 2 * (u.t1 - u.t0);
        int2 info;
        const int slot = iter.slot_of(u, &info);
        if (tid == 0 && leader) prm.item_info[u.it] = info;
        float inv = 0.f, lse = 0.f;
        for (int pi = 0; pi < npages && ok; ++pi, ++gt) {
          const uint32_t s = gt % kNumP, k = gt / kNumP;
          ok = warp_wait<true>(bar(B_PFULL + s), k & 1);
          if (!ok) break;
          if (tid == 0) QSTAMP(smem_base, 6, gt);
          const uint32_t pbuf = smem_base + kOffP + s * kPStride;
          const uint32_t nword = ld_shared_b32(pbuf + kNOff + r * 4);
          if (pi + 1 == npages) {
            uint32_t x, y;
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(pbuf + kFinOff + r * 8));
            inv = __uint_as_float(x); lse = __uint_as_float(y);
          }
          const bool mine = (kMode == 2) ? (__uint_as_float(nword) != 1.f) : (nword != 0u);
          if (__any_sync(0xffffffffu, mine) && pi > 0) {
            // lines 13-16: O <- AS_FP32(AS_INT32(O) + N), after P V of the previous page has landed
            const uint32_t gp = gt - 1;
            ok = warp_wait(bar(X_PV + gp % kNumP), (gp / kNumP) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            auto apply = [&](uint32_t (&o)[32]) {
              if (kMode == 2) {
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * __uint_as_float(nword));
              } else if (!kGuard) {
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(exponent_add_raw(__uint_as_float(o[i]), static_cast<int>(nword)));
              } else {
                // the guard matters only where magnitude bits + N would not stay positive: take the chunk's smallest
                // magnitude first and use the plain one-instruction add of Lemma 3.1 where it is safe
                float lo = fmin3_abs(__uint_as_float(o[0]), __uint_as_float(o[1]), __uint_as_float(o[2]));
#pragma unroll
                for (int i = 3; i + 1 < 32; i += 2) lo = fmin3_abs(lo, __uint_as_float(o[i]), __uint_as_float(o[i + 1]));
                lo = fminf(lo, fabsf(__uint_as_float(o[31])));
                if (__float_as_int(lo) + static_cast<int>(nword) > 0) {
#pragma unroll
                  for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(exponent_add_raw(__uint_as_float(o[i]), static_cast<int>(nword)));
                } else {
#pragma unroll
                  for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(exponent_add_guarded(__uint_as_float(o[i]), static_cast<int>(nword)));
                }
              }
            };
            uint32_t o0[32], o1[32];
            const uint32_t obase = tbase + lane_base + 32 * c_first;
            tmem_ld_32x32b_x32(obase, o0);
#pragma unroll 1
            for (int cc = 0; cc < 8; cc += 2) {
              tmem_wait_ld();
              tmem_ld_32x32b_x32(obase + 32 * (cc + 1), o1);
              apply(o0);
              tmem_st_32x32b_x32(obase + 32 * cc, o0);
              tmem_wait_ld();
              if (cc + 2 < 8) tmem_ld_32x32b_x32(obase + 32 * (cc + 2), o0);
              apply(o1);
              tmem_st_32x32b_x32(obase + 32 * (cc + 1), o1);
            }
            tmem_wait_st();
            tc_fence_before_sync();
          }
          warp_arrive(bar(B_OREADY + s), lane);
          if (tid == 0) QSTAMP(smem_base, 7, gt);
        }
        if (!ok) break;
        // ---- epilogue (line 20): out = O / (l * S16).  Thread = row; a warp and its partner take eight 32-column
        // chunks each, scale them and store them from registers with 256-bit stores (a full 32-byte sector per lane).
        {
          const uint32_t gl = gt - 1;
          if (tid == 0) QSTAMP(smem_base, 14, un);
          ok = warp_wait(bar(X_PV + gl % kNumP), (gl / kNumP) & 1);
          if (!ok) break;
          tc_fence_after_sync();
          if (tid == 0) { QSTAMP(smem_base, 12, un); if (un < 1) QSTAMP_NS(smem_base, 3); };
          const int row = u.r0 + half * kRowBlock + r;               // this thread's row within the sequence
          const bool valid = row < prm.R;
          __nv_bfloat16* orow = prm.out + (static_cast<size_t>(u.b) * prm.R + (valid ? row : 0)) * kDv;
          const size_t prow = static_cast<size_t>(slot < 0 ? 0 : slot) * kItemRows + half * kRowBlock + r;   // row of the partial arrays
          uint16_t* hrow = partial_halves(prm) + prow * kDv;
          uint32_t sc_lo = 0, sc_hi = 0;                                  // this thread's eight scale bytes
          uint32_t o[2][32];
          tmem_ld_32x32b_x32(tbase + lane_base + 32 * c_first, o[0]);
#pragma unroll 1
          for (int cq = 0; cq < 8; cq += 2) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              tmem_wait_ld();
              if (cq + e + 1 < 8) tmem_ld_32x32b_x32(tbase + lane_base + 32 * (c_first + cq + e + 1), o[e ^ 1]);
              const int cc = c_first + cq + e;
              uint32_t w[16];
              uint16_t* dst;
              if (slot < 0) {
                epilogue_chunk_bf16(o[e], inv, w);
                dst = reinterpret_cast<uint16_t*>(orow) + 32 * cc;
              } else {
                const uint32_t sb = epilogue_chunk_partial(o[e], inv, w);
                if (cq + e < 4) sc_lo |= sb << (8 * (cq + e)); else sc_hi |= sb << (8 * (cq + e - 4));
                dst = hrow + 32 * cc;
              }
              if (valid) {
                stg_256(dst, w[0], w[1], w[2], w[3], w[4], w[5], w[6], w[7]);
                stg_256(dst + 16, w[8], w[9], w[10], w[11], w[12], w[13], w[14], w[15]);
              }
            }
          }
          if (valid && slot >= 0)
            *reinterpret_cast<uint2*>(partial_scales(prm) + prow * 16 + c_first) = make_uint2(sc_lo, sc_hi);
          if (valid && !partner) {
            if (slot < 0) prm.lse[static_cast<size_t>(u.b) * prm.R + row] = lse;
            else prm.part_lse[prow] = lse;
          }
          tc_fence_before_sync();
          if (tid == 0) QSTAMP(smem_base, 13, un);
        }
        ++un;
      }
      if (!ok) report_timeout(prm.status);
    } else if (wid == 4) {
      // ---- TMA producers: V.  One slot per page: this CTA's 128 columns of either 256-column half of V (two
      // boxes of 64 keys x 128 columns); lane l owns ring slot l.  Both pages of every tile are loaded (the
      // second page of a sequence's odd last tile is the first one again; its probabilities are zero).
      Cursor cur(prm, prefix, seqlens, part);
      int my_gp = lane;                       // next page of the sequence this lane loads (tile = gp / 2)
      uint32_t par = 1;
      bool fin = lane >= kNumVSlots, have = false;
      int page_id = 0;
      int issued = 0;
      const uint32_t my_full = bar(B_VFULL + lane), my_empty = bar(B_VEMPTY + lane);
      const uint32_t lead_full = lead_bars + 8u * (B_VFULL + lane);
      const uint32_t dst = smem_base + kOffV + lane * kVSlotBytes;
      uint64_t t_start = global_timer_ns();
      bool progress = false;
      for (uint32_t spin = 0;; ++spin) {
        if (!fin && !have) {
          int lt;
          if (cur.locate(my_gp >> 1, lt)) {
            const int t = cur.u.t0 + lt;
            const int npg = (cur.u.n_b + kPage - 1) / kPage;
            const int pg = (2 * t + (my_gp & 1) < npg) ? 2 * t + (my_gp & 1) : 2 * t;
            page_id = __ldg(prm.block_table + static_cast<size_t>(cur.u.b) * prm.max_blocks_per_seq + pg);
            have = true;
          } else {
            fin = true;
          }
        }
        if (have && mbar_probe(my_empty, par)) {
          if (leader) mbar_arrive_expect_tx(my_full, 2 * kVSlotBytes);
          tma_load_3d_pair(dst, &v_map, 0, page_id * kPage, 2 * half, lead_full);
          tma_load_3d_pair(dst + kVHalfBytes, &v_map, 0, page_id * kPage, 4 + 2 * half, lead_full);
          my_gp += kNumVSlots;
          par ^= 1;
          ++issued;
          have = false;
          progress = true;
        }
        if (__all_sync(0xffffffffu, fin)) break;
        const bool any_progress = __any_sync(0xffffffffu, progress);
        if (any_progress) t_start = global_timer_ns(); else __nanosleep(100);
        progress = false;
        if ((spin & 1023u) == 1023u && __any_sync(0xffffffffu, global_timer_ns() - t_start > kWaitLimitNs)) { ok = false; break; }
      }
      if (!ok) {
        if (lane == 0) report_timeout(prm.status);
        if (leader && issued > 0 && lane < kNumVSlots) mbar_wait(my_full, (issued - 1) & 1);
      }
    } else if (wid == 5) {
      // ---- MMA issuer (even CTA only): O (+)= P~ V for both CTAs' rows; per page two N = 256 halves of four
      // K = 16 steps
      if (leader && lane == 0) {
        constexpr uint32_t idesc = make_idesc_bf16(256, 256, false, true);
        constexpr uint32_t dhi = smem_desc_hi_sw128(1024);
        const uint32_t vlo0 = smem_desc_lo(smem_base + kOffV, kBoxBytes);
        const uint32_t plo0 = smem_desc_lo(smem_base + kOffP, 16);
        uint32_t slot = 0, vpar = 0;
        while (ok && iter.next(u)) {
          const int npages = 2 * (u.t1 - u.t0);
          for (int pi = 0; pi < npages && ok; ++pi, ++gt) {
            const uint32_t s = gt % kNumP, k = gt / kNumP;
            ok = mbar_wait<true>(bar(B_PFULL + s), k & 1);
            if (!ok) break;
            QSTAMP(smem_base, 10, gt);
            ok = mbar_wait(bar(B_OREADY + s), k & 1);
            if (!ok) break;
            QSTAMP(smem_base, 11, gt);
            tc_fence_after_sync();
            fence_proxy_async_smem();
            ok = mbar_wait(bar(B_VFULL) + 8 * slot, vpar);
            if (!ok) break;
            QSTAMP(smem_base, 8, gt);
            const uint32_t plo = plo0 + s * (kPStride >> 4);
            const uint32_t vlo = vlo0 + slot * (kVSlotBytes >> 4);
            const uint32_t acc0 = pi > 0 ? 1u : 0u;
#pragma unroll
            for (int nh = 0; nh < 2; ++nh) {
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                mma_ss_pair(tbase + nh * 256, smem_desc_join(plo + 2 * kk, dhi), smem_desc_join(vlo + nh * (kVHalfBytes >> 4) + 128 * kk, dhi),
                            idesc, kk == 0 ? acc0 : 1u);
            }
            mma_commit_pair_multicast(bar(B_VEMPTY) + 8 * slot, kMaskValue);
            if (++slot == kNumVSlots) { slot = 0; vpar ^= 1; }
            mma_commit_pair_multicast(bar(X_PV + s), kMaskAll);   // PVDONE in the value CTAs, "P buffer free" in the score CTAs
            QSTAMP(smem_base, 9, gt);
          }
          if (!ok) break;
        }
        if (!ok) report_timeout(prm.status);
      } else if (!leader) {
        // ---- relay (odd CTA): lane s passes on the completed phases of OREADY[s] (the pages in P buffer s).  The
        // page's P~ in this CTA (remote asynchronous stores, generic proxy) is about to be read by the pair MMA.
        int n_pages = 0;
        while (iter.next(u)) n_pages += 2 * (u.t1 - u.t0);
        const int phases = lane < kNumP ? (n_pages + kNumP - 1 - lane) / kNumP : 0;
        if (!relay_phases<true>(bars, lead_bars, B_OREADY, lane, phases) && lane == 0) report_timeout(prm.status);
      }
    }
  }

  // teardown: nobody may still be writing into a CTA that has exited, and both CTAs of a pair must be done
  // with tensor memory before it is freed
  if (tid == 0) QSTAMP_NS(smem_base, 4);
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0) QSTAMP_NS(smem_base, 5);
#ifdef AMLA_TRACE
  if (prm.trace) {
    for (int i = tid; i < kQTraceEvents * kQTraceIdx; i += kThreads)
      prm.trace[static_cast<size_t>(blockIdx.x) * kQTraceEvents * kQTraceIdx + i] = ld_shared_b32(smem_base + kOffTrace + 4 * i);
  }
#endif
  cluster_arrive();
  cluster_wait();
#ifdef AMLA_TRACE
  if (prm.trace && tid == 0) prm.trace[static_cast<size_t>(blockIdx.x) * kQTraceEvents * kQTraceIdx + 15 * kQTraceIdx + 7] = static_cast<uint32_t>(global_timer_ns());   // idx 7 < kQTraceIdx
#endif
  if (wid == 5) tmem_dealloc_pair(tbase, kTmemCols);
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static std::atomic<EncodeTiledFn> fn{nullptr};
  EncodeTiledFn f = fn.load(std::memory_order_acquire);
  if (!f) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess) {
      f = reinterpret_cast<EncodeTiledFn>(p);
      fn.store(f, std::memory_order_release);
    }
  }
  return f;
}

void fill_config(cudaLaunchConfig_t& cfg, cudaLaunchAttribute* attr, int clusters, cudaStream_t stream) {
  cfg = cudaLaunchConfig_t{};
  cfg.gridDim = dim3(4 * clusters);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
}

template <int kMode, bool kGuard>
cudaError_t prepare_variant(int device) {
  static std::atomic<uint64_t> done{0};
  const uint64_t bit = 1ull << (device & 63);
  if (!(done.load(std::memory_order_acquire) & bit)) {
    const cudaError_t err = cudaFuncSetAttribute(decode_quad_kernel<kMode, kGuard>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemBytes));
    if (err != cudaSuccess) return err;
    done.fetch_or(bit, std::memory_order_release);
  }
  return cudaSuccess;
}

template <int kMode, bool kGuard>
cudaError_t launch_variant(const CUtensorMap& kmap, const CUtensorMap& vmap, const CUtensorMap& qmap, const DecodeParams& prm, cudaStream_t stream) {
  int device = 0;
  cudaError_t err = cudaGetDevice(&device);
  if (err != cudaSuccess) return err;
  err = prepare_variant<kMode, kGuard>(device);
  if (err != cudaSuccess) return err;
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  fill_config(cfg, attr, prm.P, stream);
  return cudaLaunchKernelEx(&cfg, decode_quad_kernel<kMode, kGuard>, kmap, vmap, qmap, prm);
}

}  // namespace

// Number of four-CTA clusters that can be resident at once on `device` (0 if the query fails): the parts the
// schedule is cut into.  Queried once per device.
int decode_quad_parts(int device, int sm_count) {
  static std::atomic<int> cache[64];
  if (device < 0 || device >= 64) return 0;
  int v = cache[device].load(std::memory_order_acquire);
  if (v > 0) return v;
  if (prepare_variant<0, true>(device) != cudaSuccess) { cudaGetLastError(); return 0; }
  cudaLaunchConfig_t cfg;
  cudaLaunchAttribute attr[1];
  fill_config(cfg, attr, sm_count / 4 > 0 ? sm_count / 4 : 1, nullptr);
  cfg.numAttrs = 0;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, decode_quad_kernel<0, true>, &cfg) != cudaSuccess || n <= 0) { cudaGetLastError(); return 0; }
  if (n > sm_count / 4) n = sm_count / 4;
  cache[device].store(n, std::memory_order_release);
  return n;
}

cudaError_t launch_decode_quad(const DecodeParams& prm, cudaStream_t stream, int* unsupported) {
  *unsupported = 0;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) { *unsupported = 1; return cudaErrorNotSupported; }
  // K: the cache seen as (64 columns, 8 rows of a group, 9 column blocks, row groups); one box = a page's 64 keys x
  // 3 column blocks, laid out in shared memory as [row group][column block][8 keys][64 columns], so that a
  // K-major operand descriptor with a group stride of 3 KB walks the keys of one column block.
  CUtensorMap kmap;
  {
    const cuuint64_t dims[4] = {64, 8, static_cast<cuuint64_t>(kDqk / 64), static_cast<cuuint64_t>(prm.num_blocks) * 8};
    const cuuint64_t strides[3] = {static_cast<cuuint64_t>(kDqk) * 2, 128, static_cast<cuuint64_t>(kDqk) * 2 * 8};
    const cuuint32_t box[4] = {64, 8, 3, 8};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult cr = encode(&kmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(prm.kv), dims, strides,
                               box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  // V: the same rows seen as (64 columns, rows, column block); one box = 64 keys x 2 column blocks, laid out in
  // shared memory as [column block][key][64 columns]: the MN-major B operand of 128 output columns.
  CUtensorMap vmap;
  {
    const cuuint64_t vdims[3] = {64, static_cast<cuuint64_t>(prm.num_blocks) * kPage, static_cast<cuuint64_t>(kDqk / 64)};
    const cuuint64_t vstrides[2] = {static_cast<cuuint64_t>(kDqk) * 2, 128};
    const cuuint32_t vbox[3] = {64, 64, 2};
    const cuuint32_t vestr[3] = {1, 1, 1};
    const CUresult vr = encode(&vmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(prm.kv), vdims, vstrides,
                               vbox, vestr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (vr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  // Q: (64 columns, rows of all sequences, 9 column blocks); one box = 64 rows x one column block, laid out
  // [row][64 columns] like an operand tile.  Rows past the end of the array read as zero; rows of a following
  // sequence that a short block's boxes cover are dropped by the kernel.
  CUtensorMap qmap;
  {
    const cuuint64_t qdims[3] = {64, static_cast<cuuint64_t>(prm.B) * prm.R, static_cast<cuuint64_t>(kDqk / 64)};
    const cuuint64_t qstrides[2] = {static_cast<cuuint64_t>(kDqk) * 2, 128};
    const cuuint32_t qbox[3] = {64, 64, 1};
    const cuuint32_t qestr[3] = {1, 1, 1};
    const CUresult qr = encode(&qmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(prm.q), qdims, qstrides,
                               qbox, qestr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (qr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  const int mode = prm.flags & 3;
  const bool guard = !(prm.flags & 4);
  if (mode == 0) return guard ? launch_variant<0, true>(kmap, vmap, qmap, prm, stream) : launch_variant<0, false>(kmap, vmap, qmap, prm, stream);
  if (mode == 1) return guard ? launch_variant<1, true>(kmap, vmap, qmap, prm, stream) : launch_variant<1, false>(kmap, vmap, qmap, prm, stream);
  return launch_variant<2, true>(kmap, vmap, qmap, prm, stream);
}

}  // namespace amla

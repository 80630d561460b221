// Tensor-core MLA decode kernel for sm_100a.
//
// A cluster of two CTAs works on one 128-row block of query rows and a range of 64-key cache pages:
//
//   score CTA (cluster rank 0)   the 512 latent columns of Q (128 x 512 bf16) are resident in tensor
//       memory as the A operand, the 64 RoPE columns in shared memory.  K arrives by TMA in slots of
//       128 keys x 192 columns (two pages stacked, one 4-D box each), three slots per score tile,
//       through a ring; S = Q K^T (128 x 128, FP32) by tcgen05.mma into a double-buffered TMEM tile.  The
//       softmax warpgroup runs Algorithm 2's per-row recurrence (lines 5-12) once per score tile,
//       writes the bf16 probabilities P~ = bf16(P * S16) of each 64-key half plus the per-row integer
//       N into a local staging buffer, and four copy warps move it into the value CTA with
//       asynchronous remote stores counted on a barrier there.
//   value CTA (cluster rank 1)   the whole FP32 accumulator O (128 x 512) lives in its tensor memory;
//       V (first 512 columns of the same cache rows) arrives by TMA in slots of 64 keys x 256
//       columns through a 4-slot ring; a correction warpgroup applies N to the bit patterns of O
//       (lines 13-16; Lemma 3.1) for rows whose reference moved, then O += P~ V by tcgen05.mma
//       (lines 17-18); the epilogue divides by l * S16 (line 20).
//
// This is the counterpart of the paper's split between matrix and vector units (Section 3.3) with
// its [C1, C2, V1] steady-state order (Section 4.1): QK^T of the next tile is issued before P V of
// this one finishes, and the softmax overlaps both.  What differs: O never leaves tensor memory, so
// the integer add is a TMEM load/add/store rather than an atomic in global memory.
//
// All waits are bounded; on expiry the kernel records kStatusTimeout and unwinds.
#include <atomic>
#include <type_traits>

#include "amla_common.cuh"
#include "amla_sm100.cuh"
#include "amla_epilogue.cuh"

namespace amla {

using namespace sm100;

// trace builds: wall-clock stamps (global timer, ns) of a CTA's phases, in event row 31, columns 88..95
#ifdef AMLA_TRACE
#define AMLA_STAMP_NS(prm, part, col)                                                                               \
  do {                                                                                                              \
    if ((prm).trace) (prm).trace[(static_cast<size_t>(part) * kTraceEvents + 31) * kTraceTiles + (col)] = global_timer_ns(); \
  } while (0)
#else
#define AMLA_STAMP_NS(prm, part, col) do { } while (0)
#endif

namespace {

constexpr int kNumCopyWarps = 4;         // score CTA: warps that move staged P~ to the value CTA
#ifdef AMLA_TRACE
constexpr int kThreads = 32 * (7 + kNumCopyWarps);   // trace builds add a last warp, which watches the K slots fill
#else
constexpr int kThreads = 32 * (6 + kNumCopyWarps);   // warps 0-3: softmax / correction, 4: TMA producers, 5: MMA issuer + TMEM alloc, 6..: P copy
#endif
constexpr uint32_t kBoxBytes = 64 * 64 * 2;             // one 64-key x 64-column TMA box
constexpr uint32_t kPBytes = 128 * 64 * 2;              // P~ of one 64-key half: 128 rows x 128 B
constexpr uint32_t kPXfer = kPBytes + 128 * 4;          // ... followed by the 128 per-row integers
constexpr uint32_t kPStride = 17 * 1024;                // distance between P buffers
constexpr int kNumP = 4;                                // P buffers in the value CTA (pages the softmax may run ahead)

// ---- score CTA
constexpr int kNumKSlots = 4;                           // 192 KB in flight: what the load latency needs at the MMA's rate
constexpr uint32_t kKPageBytes = 3 * kBoxBytes;         // 64 keys x 3 column blocks: [8 row groups][3 blocks][8 rows][128 B]
constexpr uint32_t kKSlotBytes = 2 * kKPageBytes;       // 128 keys x 192 columns (two pages stacked)
constexpr uint32_t kKGroupStride = 3 * 1024;            // distance between 8-row groups inside a slot
constexpr uint32_t kOffQRope = 0;                       // 128 rows x 64 bf16, 128-byte swizzle
constexpr uint32_t kOffStage = 128 * 64 * 2;            // kPStride: P~ and N of a page, before the copy warps move them to the value CTA
constexpr uint32_t kOffK = kOffStage + kPStride;
constexpr uint32_t kEndA = kOffK + kNumKSlots * kKSlotBytes;
// ---- value CTA
constexpr int kNumVSlots = 4;
constexpr uint32_t kVSlotBytes = 4 * kBoxBytes;         // 64 keys x 256 columns
constexpr uint32_t kOffV = 0;
constexpr uint32_t kOffP = kNumVSlots * kVSlotBytes;    // kNumP x kPStride (P~ then N)
constexpr uint32_t kOffFin = kOffP + kNumP * kPStride;  // float2 [2][128] (1/(l*S16), lse)
constexpr uint32_t kEndB = kOffFin + 2 * 128 * 8;
// ---- both: the barriers sit at the same offset, so that one multicast commit can reach the two CTAs
constexpr uint32_t kOffBars = kEndA > kEndB ? kEndA : kEndB;
constexpr uint32_t kBarBytes = 512;
// ---- both: a copy of the schedule prefix and of the sequence lengths for batches of up to kSmemPlanItems items,
// so that the roles' schedule look-ups (a dozen dependent loads per unit) stay on chip
constexpr int kSmemPlanItems = 128;
constexpr uint32_t kOffPlan = kOffBars + kBarBytes;                          // int [kSmemPlanItems + 1] prefix
constexpr uint32_t kOffSeqlens = kOffPlan + ((kSmemPlanItems + 1) * 4 + 15) / 16 * 16;   // int [kSmemPlanItems] sequence lengths
constexpr uint32_t kSmemBytes = kOffSeqlens + kSmemPlanItems * 4;
static_assert(kSmemBytes <= 232448, "exceeds the shared memory a block can opt in to");
static_assert(kOffK % 1024 == 0 && kOffP % 1024 == 0, "swizzled tiles need 1024-byte alignment");

// tensor-memory columns
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kQCol = 0;            // score CTA: latent part of Q, 256 columns (two bf16 per column)
constexpr uint32_t kSCol = 256;          // score CTA: S buffers, 2 x 128 columns
// value CTA: O occupies columns 0..511

// Barrier indices.  X_PV is shared: in the value CTA it completes when P V of a page has finished (PVDONE), in the
// score CTA the same arrival (multicast commit) frees the page's P buffer for the softmax (PEMPTY).
enum { X_PV = 0, X_COMMON = X_PV + kNumP };
enum { A_KFULL = X_COMMON, A_KEMPTY = A_KFULL + kNumKSlots, A_SFULL = A_KEMPTY + kNumKSlots, A_SEMPTY = A_SFULL + 2,
       A_PSTAGED = A_SEMPTY + 2, A_STAGEFREE = A_PSTAGED + 2, A_QREADY = A_STAGEFREE + 2, A_QFREE, A_FINFREE, A_QDONE = A_FINFREE + 2, A_NUM = A_QDONE + kNumKSlots };
enum { B_VFULL = X_COMMON, B_VEMPTY = B_VFULL + kNumVSlots, B_PFULL = B_VEMPTY + kNumVSlots, B_OREADY = B_PFULL + kNumP,
       B_FINFULL = B_OREADY + kNumP, B_NUM = B_FINFULL + 2 };
static_assert(A_NUM * 8 + 8 <= kBarBytes && B_NUM * 8 + 8 <= kBarBytes, "barrier area too small");

struct Unit {
  int b, r0, nrows, n_b, t0, t1, it;
};

// Walks the (part, item) intersections of this cluster's part in schedule order.
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
      if (hi > lo) { u.t0 = lo - a; u.t1 = hi - a; break; }   // else: only overhead positions of this item fell into the part
    }
    u.it = it;
    u.b = it / prm.nrb;
    u.r0 = (it % prm.nrb) * kRowBlock;
    u.nrows = min(kRowBlock, prm.R - u.r0);
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

// Finds the unit that holds the k-th page (kTiles = false) or the k-th score tile (kTiles = true) of this
// cluster's part; k never decreases between calls.  Used by producer lanes that advance independently.
template <bool kTiles>
struct Cursor {
  UnitIter it;
  Unit u;
  int base;      // index of the current unit's first page / score tile
  int ord;       // ordinal of the current unit within the part
  bool valid;
  __device__ Cursor(const DecodeParams& prm, const int* prefix, const int* seqlens, int part) : it(prm, prefix, seqlens, part), base(0), ord(0) { valid = it.next(u); }
  // adopts a walk whose first unit (`first`, if `has_first`) has been looked up already
  __device__ Cursor(const UnitIter& after_first, const Unit& first, bool has_first) : it(after_first), u(first), base(0), ord(0), valid(has_first) {}
  __device__ int count() const { return kTiles ? (u.t1 - u.t0 + 1) / 2 : (u.t1 - u.t0); }
  // false when k lies beyond the part's work; otherwise `local` is the index within the unit
  __device__ bool locate(int k, int& local) {
    while (valid && k >= base + count()) { base += count(); valid = it.next(u); ++ord; }
    local = k - base;
    return valid;
  }
};

__device__ __forceinline__ void report_timeout(int* status) { atomicExch(status, kStatusTimeout); }

// Wait whose verdict is the same in every lane of the warp, so that the warp-collective tensor-memory
// instructions that follow are never executed by a part of it.
template <bool kClusterAcquire = false>
__device__ __forceinline__ bool warp_wait(uint32_t bar, uint32_t parity) {
  return __all_sync(0xffffffffu, mbar_wait<kClusterAcquire>(bar, parity));
}

// Brings the nine 128-byte lines of one query row of a unit into L2 ahead of the loads that move it on chip.
__device__ __forceinline__ void prefetch_q_row(const DecodeParams& prm, const Unit& u, int row) {
  if (row < u.nrows) {
    const char* p = reinterpret_cast<const char*>(prm.q + (static_cast<size_t>(u.b) * prm.R + u.r0 + row) * kDqk);
#pragma unroll
    for (int i = 0; i < 9; ++i) prefetch_l2(p + 128 * i);
  }
}

// Q comes on chip through the K ring: at the start of a unit every ring slot takes two 64-column blocks of the unit's
// 128 rows (TMA boxes, [block][row][128 B] with the 128-byte swizzle), the RoPE block goes straight to its operand tile.
// Eight warps then move the latent blocks into tensor memory: thread = row, a warp and its partner take one block of
// the slot each.  This is one block: 128 bytes of the row from the swizzled box into 32 columns (two bf16 per column).
constexpr uint32_t kQBlockBytes = 128 * 128;            // one 64-column block of 128 rows
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

// The eight Q warps' share of a unit's start: wait for each slot's piece, move it, hand the slot back.  `gs` = score
// tiles of this cluster before the unit (three K slots each), `un` = units before it: slot e has completed
// un + ceil((3 gs - e) / 4) phases so far.  Returns false after a timeout.
__device__ __forceinline__ bool move_q_unit(const DecodeParams& prm, int part, uint32_t smem_base, uint32_t bars, uint32_t taddr_row, int row, bool valid, int blk,
                                            uint32_t un, uint32_t gs, int lane) {
  bool ok = true;
#pragma unroll 1
  for (int e = 0; e < kNumKSlots && ok; ++e) {
    const uint32_t par = (un + (3 * gs + 3 - e) / 4) & 1;
    ok = __all_sync(0xffffffffu, mbar_wait(bars + 8u * (A_KFULL + e), par));
    if (!ok) break;
    if (row == 0) AMLA_STAMP2(prm, part, 28 + blk, un * kNumKSlots + e);
    move_q_block(smem_base + kOffK + e * kKSlotBytes + blk * kQBlockBytes, row, valid, taddr_row + 32 * (2 * e + blk));
    __syncwarp();                                       // every lane's reads of the slot are done
    if (lane == 0) mbar_arrive(bars + 8u * (A_QDONE + e));
  }
  return ok;
}

// What a role needs from the kernel's set-up.
struct RoleCtx {
  uint32_t smem_base, bars, tbase, peerB_bars, peerB_base;
  const int* prefix;
  const int* seqlens;
  int part, tid;
};

// The softmax warpgroup's work on one unit: its score tiles, then the final scalars for the value CTA.  A function
// of its own, so that it can also be run and timed outside the kernel.  Returns
// (pages so far) << 32 | (score tiles so far) << 1 | ok.
template <int kMode>
__device__ __noinline__ uint64_t softmax_unit(const DecodeParams prm, const RoleCtx c, const Unit u, uint32_t un, uint32_t gt, uint32_t gs) {
  const int tid = c.tid, wid = tid >> 5, part = c.part;
  const uint32_t smem_base = c.smem_base, bars = c.bars, tbase = c.tbase, peerB_bars = c.peerB_bars, peerB_base = c.peerB_base;
  auto bar = [&](int i) { return bars + 8u * i; };
  (void)part;
  bool ok = true;
  const int r = tid;
  const uint32_t lane_base = static_cast<uint32_t>(wid * 32) << 16;
  const bool scale_nonneg = prm.scale_log2 >= 0.f;
  const uint32_t mask_fill = __float_as_uint(scale_nonneg ? -INFINITY : INFINITY);
  {
    RowState st;
    row_state_init(st);
    const int tok = (u.r0 + r) / prm.H;
    const int visible = min(u.n_b, u.n_b - prm.Sq + tok + 1);          // keys 0..visible-1 are seen by this row
    const int first_masked_tile = max(u.n_b - prm.Sq + 1, 0) / kPage;  // pages from here on may hold hidden keys

    for (int t = u.t0; t < u.t1 && ok; t += 2, ++gs) {
      const int npages = min(2, u.t1 - t);
      const uint32_t sb = gs & 1;
      ok = warp_wait(bar(A_SFULL + sb), (gs >> 1) & 1);
      if (!ok) break;
      tc_fence_after_sync();
      if (tid == 0) AMLA_STAMP(prm, part, 5, gt);
      const uint32_t scol = tbase + lane_base + kSCol + 128 * sb;
      const int nvis = visible - t * kPage;              // keys of this score tile the row sees (may be <= 0)
      // Two compilations of the tile: the plain one (every key visible, non-negative scale), and the general one
      // with the visibility masks and the sign of the scale; a run-time flag inside one body costs the plain
      // tiles their instruction schedule.
      auto tile_body = [&](auto general_c) {
      constexpr bool kGeneral = decltype(general_c)::value;
      constexpr bool masked = kGeneral;
      const bool scale_nn = kGeneral ? scale_nonneg : true;

      // The S tile is read from tensor memory in 32-column chunks, twice (maximum, then exponentials); the load
      // of the next chunk is always in flight while a chunk is processed, so that the TMEM latency is hidden.
      uint32_t b0[32], b1[32];
      // lines 5-6: running max, taken on the raw scores (the scale is folded into the FMA below)
      float ext = scale_nn ? -INFINITY : INFINITY, ext_b = ext;      // two chains: half the dependent latency
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
      tmem_ld_32x32b_x32(scol, b0);
#pragma unroll 1
      for (int h = 0; h < npages; ++h) {
        tmem_wait_ld();
        tmem_ld_32x32b_x32(scol + 64 * h + 32, b1);
        chunk_max(b0, 64 * h);
        tmem_wait_ld();
        tmem_ld_32x32b_x32(scol + (h + 1 < npages ? 64 * (h + 1) : 0), b0);   // next half, or the first chunk again for the second pass
        chunk_max(b1, 64 * h + 32);
      }
      ext = scale_nn ? fmaxf(ext, ext_b) : fminf(ext, ext_b);
      const float tmax = (nvis > 0) ? ext * prm.scale_log2 : -INFINITY;
      // Lazy reference: a row must move when its maximum exceeds the reference by more than tau.  The correction warp
      // that serves these 32 rows pays for a rescale as soon as one of them moves, so when one must, every row of the
      // warp whose maximum rose moves with it (moving early is always allowed: tau = 0 moves at every rise); the rows
      // then tend to stay in step and the warp rescales on far fewer tiles.
      const bool must = tmax > st.m2 + prm.tau;
      const RowStep sp = row_step<kMode>(st, tmax, __any_sync(0xffffffffu, must) ? 0.f : prm.tau);
      // Line 10's factor S16 goes into the exponential's argument (the paper's remark after Algorithm 2):
      // P * S16 = 2^(a - m + log2 S16).  The row sum of line 6 is the sum of the same FP32 values, taken
      // before the bf16 cast and divided by S16 once per tile.
      const float nsub = log2f_approx(sp.p_scale) - sp.m2_sub;
      float rs0 = 0.f, rs1 = 0.f;
      const uint64_t sc2 = pack_f32x2(prm.scale_log2, prm.scale_log2), ns2 = pack_f32x2(nsub, nsub);
      uint64_t rsa = pack_f32x2(0.f, 0.f), rsb = rsa;
      uint32_t pk[32];
      // lines 6, 10 for 32 columns: P, row sum (FP32, unscaled), P~ = bf16(P * S16), two elements per instruction
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
#pragma unroll 1
      for (int h = 0; h < npages; ++h) {
        tmem_wait_ld();
        tmem_ld_32x32b_x32(scol + 64 * h + 32, b1);
        chunk_exp(b0, 64 * h, 0);
        tmem_wait_ld();
        if (h + 1 < npages) {
          tmem_ld_32x32b_x32(scol + 64 * (h + 1), b0);
        } else {                       // the score tile has been read for the last time
          tc_fence_before_sync();
          mbar_arrive(bar(A_SEMPTY + sb));
          if (tid == 0) AMLA_STAMP2(prm, part, 6, gt);
        }
        // One staging buffer: the copy warps of the previous page must have read it into registers.  The barrier is
        // probed here, ahead of the last chunk's arithmetic, so that the probe's latency is not exposed (this warp
        // is alone on its scheduler); the blocking wait runs only if the probe came too early.
        const bool stage_free = gt == 0 || mbar_probe(bar(A_STAGEFREE + ((gt - 1) & 1)), ((gt - 1) >> 1) & 1);
        chunk_exp(b1, 64 * h + 32, 16);
        // stage P~ and N; the copy warps ship them to the value CTA
        const uint32_t s2 = gt & 1;
        if (tid == 0) AMLA_STAMP2(prm, part, 7, gt);
        if (!__all_sync(0xffffffffu, stage_free)) ok = warp_wait(bar(A_STAGEFREE + ((gt - 1) & 1)), ((gt - 1) >> 1) & 1);
        if (!ok) break;
        if (tid == 0) AMLA_STAMP2(prm, part, 8, gt);
        const uint32_t stg = smem_base + kOffStage;
#pragma unroll
        for (int c = 0; c < 8; ++c)
          st_shared_v4(stg + sw128_offset(r, c), pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
        // the rescale (if any) belongs to the first half; the second half leaves O alone
        const uint32_t nword = (kMode == 2) ? __float_as_uint(h == 0 ? sp.l_up : 1.f)
                                            : static_cast<uint32_t>(h == 0 ? sp.n_bits : 0);
        st_shared_b32(stg + kPBytes + r * 4, nword);
        mbar_arrive(bar(A_PSTAGED + s2));
        if (tid == 0) AMLA_STAMP(prm, part, 9, gt);
        ++gt;
      }
      {
        float s0, s1;
        unpack_f32x2(add_f32x2(rsa, rsb), s0, s1);
        rs0 += s0; rs1 += s1;
      }
      st.l = st.l * sp.l_up + __fdividef(rs0 + rs1, sp.p_scale);
      };
      if (t + npages > first_masked_tile || !scale_nonneg) tile_body(std::true_type{});
      else tile_body(std::false_type{});
    }
    // line 20 scalars: 1 / (l * S16) and lse = m + ln l
    // The two-entry buffer of the value CTA is written for unit `un` only after the epilogue of unit un - 2 has read
    // its entry (nothing else keeps this warpgroup from running two short units ahead of the epilogue).
    if (ok) ok = warp_wait<true>(bar(A_FINFREE + (un & 1)), ((un >> 1) & 1) ^ 1);
    if (ok) {
      const bool live = st.l > 0.f;
      const float inv = live ? prm.out_scale / (st.l * st.s_out) : 0.f;
      const float lse = live ? (st.m2 + log2f(st.l)) * kLn2 : -INFINITY;
      // asynchronous remote stores counted on the barrier: no thread has to wait for a cluster-scope release
      const uint32_t fdst = peerB_base + kOffFin + ((un & 1) * 128 + r) * 8;
      const uint32_t fbar = peerB_bars + 8u * (B_FINFULL + (un & 1));
      if (tid == 0) mbar_arrive_expect_tx_cluster(fbar, 128 * 8);
      st_async_v2(fdst, __float_as_uint(inv), __float_as_uint(lse), fbar);
    }
  }
  return (static_cast<uint64_t>(gt) << 32) | (static_cast<uint64_t>(gs) << 1) | (ok ? 1u : 0u);
}

}  // namespace

template <int kMode, bool kGuard>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
decode_tc_kernel(const __grid_constant__ CUtensorMap kv_map, const __grid_constant__ CUtensorMap v_map, const __grid_constant__ CUtensorMap q_map,
                 const DecodeParams prm) {
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  const uint32_t smem_base = smem_u32(smem_raw);
  const int tid = threadIdx.x, wid = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_ctarank();
  const bool is_score = rank == 0;
  const int part = blockIdx.x >> 1;
  if (smem_base & 1023u) {   // the swizzled tiles assume a 1024-byte aligned window; identical in both CTAs
    if (tid == 0) report_timeout(prm.status);
    return;
  }

  if (tid == 0) AMLA_STAMP_NS(prm, part, is_score ? 88 : 92);        // entry
  const uint32_t bars = smem_base + kOffBars;
  auto bar = [&](int i) { return bars + 8u * i; };
  const uint32_t tmem_slot = bars + kBarBytes - 8;
  // addresses of the peer's barriers / buffers (same dynamic-smem base in both CTAs)
  const uint32_t peerB_bars = map_to_cta(smem_base + kOffBars, 1);
  const uint32_t peerB_base = map_to_cta(smem_base, 1);
  const uint32_t peerA_bars = map_to_cta(smem_base + kOffBars, 0);

  // The lengths of the first 32 items are requested before anything else, so that their latency runs under the set-up
  // below (they are inputs of the call: no kernel that this one may overlap with writes them).
  int early_len = 0;
  if (wid == 6 && prm.fused_plan && lane < prm.n_items) early_len = prm.seqlens[lane / prm.nrb];
  if (tid == 0) {
    for (int i = 0; i < kNumP; ++i) mbar_init(bar(X_PV + i), 1);
    if (is_score) {
      for (int i = 0; i < kNumKSlots; ++i) { mbar_init(bar(A_KFULL + i), 1); mbar_init(bar(A_KEMPTY + i), 1); }
      for (int i = 0; i < 2; ++i) {
        mbar_init(bar(A_SFULL + i), 1); mbar_init(bar(A_SEMPTY + i), 128);
        mbar_init(bar(A_PSTAGED + i), 128); mbar_init(bar(A_STAGEFREE + i), 2);
      }
      mbar_init(bar(A_QREADY), 256);
      mbar_init(bar(A_QFREE), 1);
      for (int i = 0; i < kNumKSlots; ++i) mbar_init(bar(A_QDONE + i), 8);   // the eight warps that move Q on chip
      for (int i = 0; i < 2; ++i) mbar_init(bar(A_FINFREE + i), 8);   // the eight epilogue warps of the value CTA
    } else {
      for (int i = 0; i < kNumVSlots; ++i) { mbar_init(bar(B_VFULL + i), 1); mbar_init(bar(B_VEMPTY + i), 1); }
      for (int i = 0; i < kNumP; ++i) { mbar_init(bar(B_PFULL + i), 1); mbar_init(bar(B_OREADY + i), 256); }
      for (int i = 0; i < 2; ++i) mbar_init(bar(B_FINFULL + i), 1);    // one arrival that announces 128 x 8 bytes
    }
    fence_mbar_init();
    prefetch_tensormap(&kv_map);
    prefetch_tensormap(&v_map);
    prefetch_tensormap(&q_map);
  }
  if (wid == 5) { tmem_alloc(tmem_slot, kTmemCols); tmem_relinquish(); }
  tc_fence_before_sync();
  __syncthreads();
  cluster_arrive();
  cluster_wait();          // peer barriers are initialised before anyone signals them
  tc_fence_after_sync();
  const uint32_t tbase = ld_shared_b32(tmem_slot);
  if (tid == 0) AMLA_STAMP(prm, part, is_score ? 0 : 1, 0);

  // Launched with programmatic stream serialization: everything above ran while the kernel before this one on the
  // stream was still going; its results (the schedule kernel's prefix array, or the previous call's reads of the
  // workspace) are complete after this wait.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;");
  if (tid == 0) AMLA_STAMP_NS(prm, part, is_score ? 89 : 93);        // the kernel before has completed
  const int* prefix = prm.prefix;
  const int* seqlens = prm.seqlens;
  if (prm.fused_plan) {
    // Few items: every CTA computes the schedule prefix itself (all write the same values; the combine kernel
    // reads them later) instead of waiting for a one-block kernel.  Warp 6 scans 32 items at a time.  A small
    // batch's prefix and sequence lengths are also kept in shared memory, and the roles read those copies.
    int* ps = prm.n_items <= kSmemPlanItems ? reinterpret_cast<int*>(smem_raw + kOffPlan) : nullptr;
    if (wid == 6) {
      int* pw = const_cast<int*>(prm.prefix);
      int carry = 0;
      for (int base = 0; base < prm.n_items; base += 32) {
        const int it = base + lane;
        const int n_seq = it >= prm.n_items ? 0 : base == 0 ? early_len : prm.seqlens[it / prm.nrb];
        if (ps && it < prm.n_items) reinterpret_cast<int*>(smem_raw + kOffSeqlens)[it / prm.nrb] = n_seq;   // same value from every row block
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
  // Every thread walks its cluster's units; the first one is looked up once, here, and also tells the score CTA(s)
  // which Q rows to bring into L2 while the roles start.
  bool ok = true;
  UnitIter iter(prm, prefix, seqlens, part);
  Unit u;
  bool have = iter.next(u);
  // The producers' first block-table entries: brought into L1 now, ahead of the burst of Q, K and V requests that
  // starts below (a load that misses during that burst comes back thousands of cycles later, and a producer lane that
  // waits for one holds up the other lanes of its warp).
  if (wid == 4 && lane == 0 && have) {
    const int32_t* bt = prm.block_table + static_cast<size_t>(u.b) * prm.max_blocks_per_seq;
    prefetch_l1(bt + u.t0);
    prefetch_l1(bt + min(u.t0 + 32, u.t1 - 1));
  }
  // The first unit's Q is requested here, by the first thread that knows the unit: the producer lanes reach their
  // first load thousands of cycles later (their start-up code is longer and runs from a cold instruction cache).
  if (is_score && tid == 0 && have) {
    const int row = u.b * prm.R + u.r0;
    for (int l = 0; l < kNumKSlots; ++l) {
      const uint32_t full = bar(A_KFULL + l), dst = smem_base + kOffK + l * kKSlotBytes;
      mbar_arrive_expect_tx(full, (l == 0 ? 3 : 2) * kQBlockBytes);
      tma_load_3d(dst, &q_map, 0, row, 2 * l, full);
      tma_load_3d(dst + kQBlockBytes, &q_map, 0, row, 2 * l + 1, full);
      if (l == 0) tma_load_3d(smem_base + kOffQRope, &q_map, 0, row, 8, full);
    }
  }
  uint32_t gt = 0;      // 64-key pages processed by this cluster so far (all roles count identically)
  uint32_t un = 0;      // units processed so far

  if (is_score) {
    // ======================================================================= score CTA
    uint32_t gs = 0;    // score tiles (one or two pages) so far
    uint32_t gc = 0;    // K ring slots so far
    if (wid < 4) {
      // ---- softmax warpgroup: thread = query row
      const int r = tid;
      const uint32_t lane_base = static_cast<uint32_t>(wid * 32) << 16;
      const RoleCtx ctx{smem_base, bars, tbase, peerB_bars, peerB_base, prefix, seqlens, part, tid};
      for (; ok && have; have = iter.next(u)) {
        // Q row -> tensor memory / shared memory (the previous unit's QK^T must be finished with it)
        ok = warp_wait(bar(A_QFREE), (un & 1) ^ 1);
        if (!ok) break;
        tc_fence_after_sync();
        if (tid == 0) AMLA_STAMP(prm, part, 10, un);
        // this warpgroup moves the first block of every slot's piece of Q, the copy warps (idle at this point) the second
        ok = move_q_unit(prm, part, smem_base, bars, tbase + lane_base + kQCol, r, r < u.nrows, 0, un, gs, lane);
        if (!ok) break;
        tmem_wait_st();
        tc_fence_before_sync();
        mbar_arrive(bar(A_QREADY));
        if (tid == 0) AMLA_STAMP(prm, part, 11, un);
        // the unit's score tiles and its final scalars
        const uint64_t ret = softmax_unit<kMode>(prm, ctx, u, un, gt, gs);
        gt = static_cast<uint32_t>(ret >> 32);
        gs = static_cast<uint32_t>(ret & 0xffffffffu) >> 1;
        ok = (ret & 1u) != 0;
        ++un;
      }
      if (!ok) report_timeout(prm.status);
    } else if (wid == 4) {
      // ---- TMA producers.  Lane l owns ring slot l.  The slot carries, in this order: the lane's piece of Q at the
      // start of every unit (two 64-column blocks; lane 0 adds the RoPE block, which goes straight to its operand tile
      // once the previous unit's MMAs have let go of it), and every kNumKSlots-th K slot of the sequence (three slots
      // of 192 columns per score tile).  The lanes poll without blocking, so that a slot that is still in use never
      // holds up the loads of the others (one thread issuing a ring in order reaches a fraction of the rate).
      {
        // The first unit has been looked up and its Q requested before the roles split; the way to this lane's first
        // K load is kept short (no further look-up before it; the next unit's is made when it is first asked for).
        bool fin = lane >= kNumKSlots;
        const bool first_out = !fin && have;
        Cursor<true> cur(iter, u, have);
        UnitIter qit = iter;                    // walks the units whose Q this lane has not loaded:
        Unit qu;                                //   qu = the next one (valid once looked up), q_ord its ordinal
        bool q_left = false, q_stale = first_out;
        auto q_due = [&]() { if (q_stale) { q_left = qit.next(qu); q_stale = false; } return q_left; };
        int q_ord = first_out ? 1 : 0;
        int my_tile = lane / 3, g = lane % 3;   // score tile and column-block group of the next K slot this lane loads
        int k_state = 0;                        // 0: not looked up, 1: page numbers at hand, 2: no K slot left
        int k_ord = 0;
        int pending = 0;                        // 0: decide, 1: a piece of Q, 2: a K slot
        int last = first_out ? 1 : 0;           // what the slot holds now (same code): tells which barrier frees it
        int page0 = 0, page1 = 0, npages = 0;
        int nq = first_out ? 1 : 0, nk = 0;     // pieces of Q / K slots issued for this lane's slot
        const uint32_t my_full = bar(A_KFULL + lane), my_empty = bar(A_KEMPTY + lane), my_qdone = bar(A_QDONE + lane);
        const uint32_t dst = smem_base + kOffK + lane * kKSlotBytes;
        uint64_t t_start = global_timer_ns();     // restarted whenever a lane issues a load: the limit bounds one stalled wait
        bool progress = false;
        for (uint32_t spin = 0;; ++spin) {
          if (!fin && pending == 0) {
            // (the cursor's unit is never behind the unit of the next K slot: when Q is due by that count, it goes out
            // before the K slot is looked up -- the unit's first load should not wait for a block-table entry)
            if (q_ord <= cur.ord && q_due()) pending = 1;
            else if (k_state == 0) {
              int lt;
              if (cur.locate(my_tile, lt)) {
                const int t = cur.u.t0 + 2 * lt;
                const int32_t* bt = prm.block_table + static_cast<size_t>(cur.u.b) * prm.max_blocks_per_seq;
                npages = min(2, cur.u.t1 - t);
                page0 = __ldg(bt + t);
                page1 = npages > 1 ? __ldg(bt + t + 1) : 0;
                prefetch_l1(bt + min(t + 32, cur.u.t1 - 1));     // the line after this one, well before it is needed
                k_ord = cur.ord;
                if (nk == 0) AMLA_STAMP2(prm, part, 27, 64 + lane);
                k_state = 1;
              } else {
                k_state = 2;
              }
            }
            if (pending == 0) {
              if ((k_state == 2 || q_ord <= k_ord) && q_due()) pending = 1;
              else if (k_state == 1) pending = 2;
              else if (k_state == 2) fin = true;
            }
          }
          if (pending != 0) {
            // the slot's previous content has been used up: a piece of Q by the eight Q warps, a K slot by its MMAs
            bool free_now = last == 0 || (last == 1 ? mbar_probe(my_qdone, (nq - 1) & 1) : mbar_probe(my_empty, (nk - 1) & 1));
            if (free_now && pending == 1 && lane == 0 && q_ord > 0) free_now = mbar_probe(bar(A_QFREE), (q_ord - 1) & 1);
            if (free_now) {
              if (pending == 1) {
                const int row = qu.b * prm.R + qu.r0;
                AMLA_STAMP2(prm, part, 27, q_ord * kNumKSlots + lane);
                mbar_arrive_expect_tx(my_full, (lane == 0 ? 3 : 2) * kQBlockBytes);
                tma_load_3d(dst, &q_map, 0, row, 2 * lane, my_full);
                tma_load_3d(dst + kQBlockBytes, &q_map, 0, row, 2 * lane + 1, my_full);
                if (lane == 0) tma_load_3d(smem_base + kOffQRope, &q_map, 0, row, 8, my_full);
                q_stale = true;
                ++q_ord; ++nq;
                last = 1;
              } else {
                AMLA_STAMP2(prm, part, 20, nk * kNumKSlots + lane);
                mbar_arrive_expect_tx(my_full, npages * kKPageBytes);
                tma_load_4d(dst, &kv_map, 0, 0, 3 * g, page0 * 8, my_full);
                if (npages > 1) tma_load_4d(dst + kKPageBytes, &kv_map, 0, 0, 3 * g, page1 * 8, my_full);
                // kNumKSlots slots further on
                g += kNumKSlots % 3; my_tile += kNumKSlots / 3;
                if (g >= 3) { g -= 3; my_tile += 1; }
                ++nk;
                k_state = 0;
                last = 2;
              }
              pending = 0;
              progress = true;
            }
          }
          if (__all_sync(0xffffffffu, fin)) break;
          // nothing to issue right now: back off, so that the polling does not take issue slots from the warps that
          // share this scheduler
          if (__any_sync(0xffffffffu, progress)) t_start = global_timer_ns(); else __nanosleep(100);
          progress = false;
          if ((spin & 1023u) == 1023u && __any_sync(0xffffffffu, global_timer_ns() - t_start > kWaitLimitNs)) { ok = false; break; }
        }
        if (!ok) {
          if (lane == 0) report_timeout(prm.status);
          // let the copy that may still be in flight land before the CTA exits
          if (nq + nk > 0 && lane < kNumKSlots) mbar_wait(my_full, (nq + nk - 1) & 1);
        }
      }
    } else if (wid == 5) {
      // ---- MMA issuer: S[sb] = Q K^T, 36 steps of K = 16 over three slots.  One thread runs this loop, so
      // it is kept free of divisions and descriptor arithmetic: ring position, barrier addresses and the
      // low descriptor word are stepped incrementally.
      if (lane == 0) {
        constexpr uint32_t idesc128 = make_idesc_bf16(128, 128, false, false);
        constexpr uint32_t idesc64 = make_idesc_bf16(128, 64, false, false);
        constexpr uint32_t dhi = smem_desc_hi_sw128(kKGroupStride);
        constexpr uint32_t qhi = smem_desc_hi_sw128(1024);
        const uint32_t klo0 = smem_desc_lo(smem_base + kOffK, 16);
        const uint32_t qlo0 = smem_desc_lo(smem_base + kOffQRope, 16);
        uint32_t slot = 0, kpar = 0;          // ring position and the parity its "full" barrier completes next
        for (; ok && have; have = iter.next(u)) {
          ok = mbar_wait(bar(A_QREADY), un & 1);
          if (!ok) break;
          tc_fence_after_sync();
          kpar ^= 1;                          // the unit's pieces of Q have been through every slot once
          for (int t = u.t0; t < u.t1 && ok; t += 2, ++gs) {
            const int npages = min(2, u.t1 - t);
            const uint32_t idesc = npages > 1 ? idesc128 : idesc64;
            const uint32_t sb = gs & 1;
            ok = mbar_wait(bar(A_SEMPTY + sb), ((gs >> 1) & 1) ^ 1);
            if (!ok) break;
            tc_fence_after_sync();
            AMLA_STAMP(prm, part, 3, gt);
            const uint32_t d = tbase + kSCol + 128 * sb;
            // Written out per slot and column block, so that every accumulate flag, operand offset and trip count
            // is a compile-time constant: with run-time trip counts the same loop issued 25 % slower.
#pragma unroll
            for (int g = 0; g < 3; ++g) {
              AMLA_STAMP2(prm, part, 25, gc);
              ok = ok && mbar_wait(bar(A_KFULL) + 8 * slot, kpar);    // TMA data -> MMA operand: both async proxy, no fence needed
              if (ok) {
                AMLA_STAMP2(prm, part, 21, gc);
                const uint32_t klo = klo0 + slot * (kKSlotBytes >> 4);
#pragma unroll
                for (int cl = 0; cl < 3; ++cl) {
                  const int c = 3 * g + cl;
#pragma unroll
                  for (int kk = 0; kk < 4; ++kk) {
                    const uint64_t bd = smem_desc_join(klo + 64 * cl + 2 * kk, dhi);
                    if (c < 8) mma_ts(d, tbase + kQCol + 32 * c + 8 * kk, bd, idesc, (c | kk) != 0 ? 1u : 0u);
                    else mma_ss(d, smem_desc_join(qlo0 + 2 * kk, qhi), bd, idesc, 1u);   // RoPE columns: Q from shared memory
                  }
                }
                AMLA_STAMP2(prm, part, 26, gc);
                mma_commit(bar(A_KEMPTY) + 8 * slot);
                AMLA_STAMP2(prm, part, 22, gc);
              }
              ++gc;
              if (++slot == kNumKSlots) { slot = 0; kpar ^= 1; }
            }
            if (!ok) break;
            mma_commit(bar(A_SFULL + sb));
            AMLA_STAMP(prm, part, 4, gt);
            gt += npages;
          }
          if (!ok) break;
          mma_commit(bar(A_QFREE));
          ++un;
        }
        if (!ok) report_timeout(prm.status);
      }
#ifdef AMLA_TRACE
    } else if (wid == 6 + kNumCopyWarps) {
      // trace builds: lanes 4-7 stamp the phases of the S barriers (non-blocking polls)
      if (prm.trace) {
        Cursor<true> cur(prm, prefix, seqlens, part);
        int total = 0, lt;
        while (cur.valid) { total += cur.count(); cur.locate(total, lt); }
        total *= 3;
        uint32_t par = 0;
        int gs2 = lane & 1;                       // lanes 4..7: score tile whose SFULL (4, 5) / SEMPTY (6, 7) phase comes next
        const uint64_t t_start = global_timer_ns();
        for (uint32_t spin = 0;; ++spin) {
          const bool act = false;
          const bool act2 = lane >= 4 && lane < 8 && gs2 < total / 3;
          if (act2 && mbar_probe(bar((lane < 6 ? A_SFULL : A_SEMPTY) + (lane & 1)), par)) { AMLA_STAMP2(prm, part, lane < 6 ? 30 : 31, gs2); gs2 += 2; par ^= 1; }
          if (!__any_sync(0xffffffffu, act || act2)) break;
          if ((spin & 1023u) == 1023u && __any_sync(0xffffffffu, global_timer_ns() - t_start > kWaitLimitNs)) break;
        }
      }
#endif
    } else if (wid >= 6 && wid < 6 + kNumCopyWarps) {
      // ---- copy warps: staged P~ / N of a page -> a free P buffer of the value CTA, by asynchronous remote stores
      // counted on its PFULL barrier.  (A bulk copy would queue behind the K loads in this SM's copy engine and
      // arrive thousands of cycles later; remote stores issued by the softmax threads themselves would stall them
      // at the rate of the SM-to-SM path.)  Warps c and c + 2 serve the pages of parity c -- staging buffer c --
      // and move one half of the buffer each, so every warp sees every phase of the barriers it waits on.  The
      // staging buffer is free as soon as both have read their half into registers.
      {
        const uint32_t c = (wid - 6) & 1, half = (wid - 6) >> 1;
        constexpr int kChunks = 17;                         // 512-byte chunks per warp (33 in total)
        const int qr = (wid & 3) * 32 + lane;               // query row whose second half this thread loads
        const uint32_t q_lane_base = static_cast<uint32_t>((wid & 3) * 32) << 16;
        uint32_t gs_c = 0;                                  // score tiles before the current unit
        for (; ok && have; have = iter.next(u)) {
          {
            ok = warp_wait(bar(A_QFREE), (un & 1) ^ 1);
            if (!ok) break;
            tc_fence_after_sync();
            ok = move_q_unit(prm, part, smem_base, bars, tbase + q_lane_base + kQCol, qr, qr < u.nrows, 1, un, gs_c, lane);
            if (!ok) break;
            gs_c += (u.t1 - u.t0 + 1) >> 1;
            tmem_wait_st();
            tc_fence_before_sync();
            mbar_arrive(bar(A_QREADY));
            ++un;
            UnitIter peek = iter;              // the next unit's Q goes to L2 while this one is computed
            Unit nu;
            if (peek.next(nu)) prefetch_q_row(prm, nu, qr);
          }
          for (int t = u.t0; t < u.t1; ++t, ++gt) {
            if ((gt & 1) != c) continue;
            const uint32_t pb = gt % kNumP;
            ok = warp_wait(bar(A_PSTAGED + c), (gt >> 1) & 1);
            if (!ok) break;
            const uint32_t src = smem_base + kOffStage + (half * kChunks * 32 + lane) * 16;
            uint32_t v[kChunks][4];
#pragma unroll
            for (int i = 0; i < kChunks; ++i) {
              if (half * kChunks + i < 33)
                asm volatile("ld.shared.v4.b32 {%0, %1, %2, %3}, [%4];" : "=r"(v[i][0]), "=r"(v[i][1]), "=r"(v[i][2]), "=r"(v[i][3]) : "r"(src + i * 512));
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(A_STAGEFREE + c));
            ok = warp_wait(bar(X_PV + pb), ((gt / kNumP) & 1) ^ 1);      // P V that last read the buffer is done
            if (!ok) break;
            const uint32_t pfull = peerB_bars + 8u * (B_PFULL + pb);
            const uint32_t dst = peerB_base + kOffP + pb * kPStride + (half * kChunks * 32 + lane) * 16;
            if (lane == 0 && half == 0) { AMLA_STAMP2(prm, part, 23, gt); mbar_arrive_expect_tx_cluster(pfull, kPXfer); }
#pragma unroll
            for (int i = 0; i < kChunks; ++i) {
              if (half * kChunks + i < 33) st_async_v4(dst + i * 512, v[i][0], v[i][1], v[i][2], v[i][3], pfull);
            }
          }
        }
        if (!ok && lane == 0) report_timeout(prm.status);
      }
    }
  } else {
    // ======================================================================= value CTA
    if (wid < 4 || (wid >= 6 && wid < 10)) {
      // ---- correction + epilogue warpgroup: thread = query row.  A warp reaches the tensor-memory lanes
      // 32 * (warp % 4) .. + 31, so warps 6-9, which have no other work in this CTA, are the partners of warps 2, 3,
      // 0, 1: each of a pair takes one half of the row's 512 columns, in the rescale and in the epilogue.
      const bool partner = wid >= 4;
      const int r = (wid & 3) * 32 + lane;
      const uint32_t lane_base = static_cast<uint32_t>((wid & 3) * 32) << 16;
      const int c_first = partner ? 8 : 0;          // first of this warp's eight 32-column chunks
      for (; ok && have; have = iter.next(u)) {
        int2 info;
        const int slot = iter.slot_of(u, &info);
        if (tid == 0) prm.item_info[u.it] = info;
        for (int t = u.t0; t < u.t1 && ok; ++t, ++gt) {
          const uint32_t s = gt % kNumP, k = gt / kNumP;
          ok = warp_wait<true>(bar(B_PFULL + s), k & 1);
          if (!ok) break;
          if (tid == 0) AMLA_STAMP2(prm, part, 13, gt);
          const uint32_t nword = ld_shared_b32(smem_base + kOffP + s * kPStride + kPBytes + r * 4);
          const bool mine = (kMode == 2) ? (__uint_as_float(nword) != 1.f) : (nword != 0u);
          if (__any_sync(0xffffffffu, mine) && t > u.t0) {
            // lines 13-16: O <- AS_FP32(AS_INT32(O) + N), after P V of the previous page has landed
            const uint32_t gp = gt - 1;
            ok = warp_wait(bar(X_PV + gp % kNumP), (gp / kNumP) & 1);
            if (!ok) break;
            tc_fence_after_sync();
            // two 32-column chunks in flight: the load of one overlaps the arithmetic of the other
            // The guarded add costs four integer operations per element, the FP32 multiply it replaces one.  The guard
            // only matters for an element whose magnitude bits plus N would not stay positive (an exact zero, a value
            // about to leave the normal range); so the smallest magnitude of the chunk is taken first (half an
            // operation per element), and where it is safe the chunk gets the plain one-instruction add of Lemma 3.1.
            auto apply = [&](uint32_t (&o)[32]) {
              if (kMode == 2) {
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * __uint_as_float(nword));
              } else if (!kGuard) {
#pragma unroll
                for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(exponent_add_raw(__uint_as_float(o[i]), static_cast<int>(nword)));
              } else {
                float lo = fmin3_abs(__uint_as_float(o[0]), __uint_as_float(o[1]), __uint_as_float(o[2]));
#pragma unroll
                for (int i = 3; i + 1 < 32; i += 2) lo = fmin3_abs(lo, __uint_as_float(o[i]), __uint_as_float(o[i + 1]));
                lo = fminf(lo, fabsf(__uint_as_float(o[31])));
                // NaN magnitudes compare as large numbers and take the plain add, like every other normal pattern
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
            for (int c = 0; c < 8; c += 2) {
              tmem_wait_ld();
              tmem_ld_32x32b_x32(obase + 32 * (c + 1), o1);
              apply(o0);
              tmem_st_32x32b_x32(obase + 32 * c, o0);
              tmem_wait_ld();
              if (c + 2 < 8) tmem_ld_32x32b_x32(obase + 32 * (c + 2), o0);
              apply(o1);
              tmem_st_32x32b_x32(obase + 32 * (c + 1), o1);
            }
            tmem_wait_st();
            tc_fence_before_sync();
          }
          mbar_arrive(bar(B_OREADY + s));
          if (tid == 0) AMLA_STAMP2(prm, part, 14, gt);
        }
        if (!ok) break;
        // ---- epilogue (line 20): out = O / (l * S16).  Thread = row; a warp and its partner take eight 32-column
        // chunks each, scale them and store them from registers with 256-bit stores (a full 32-byte sector per lane).  An SM
        // writes about 32 B per clock whatever the instruction: the 128 KB of a unit take 4-5 thousand clocks, and staging
        // them for tiled TMA stores (64-byte or 32-byte rows) was no faster.
        {
          const uint32_t gl = gt - 1;
          ok = warp_wait(bar(X_PV + gl % kNumP), (gl / kNumP) & 1);
          if (!ok) break;
          ok = warp_wait<true>(bar(B_FINFULL + (un & 1)), (un >> 1) & 1);
          if (!ok) break;
          tc_fence_after_sync();
          if (tid == 0) AMLA_STAMP(prm, part, 18, un);
          float inv, lse;
          {
            uint32_t x, y;
            asm volatile("ld.shared.v2.b32 {%0, %1}, [%2];" : "=r"(x), "=r"(y) : "r"(smem_base + kOffFin + ((un & 1) * 128 + r) * 8));
            inv = __uint_as_float(x); lse = __uint_as_float(y);
          }
          __syncwarp();
          if (lane == 0) mbar_arrive_cluster_relaxed(peerA_bars + 8u * (A_FINFREE + (un & 1)));   // the entry may be rewritten
          const bool valid = r < u.nrows;
          const size_t prow = static_cast<size_t>(slot < 0 ? 0 : slot) * kRowBlock + r;   // row of the partial arrays
          uint32_t sc_lo = 0, sc_hi = 0;                                  // this thread's eight scale bytes
          uint16_t* orow = reinterpret_cast<uint16_t*>(prm.out) + (static_cast<size_t>(u.b) * prm.R + u.r0 + (valid ? r : 0)) * kDv;
          uint16_t* hrow = partial_halves(prm) + prow * kDv;
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
                dst = orow + 32 * cc;
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
            if (slot < 0) prm.lse[static_cast<size_t>(u.b) * prm.R + u.r0 + r] = lse;
            else prm.part_lse[prow] = lse;
          }
          tc_fence_before_sync();
          if (tid == 0) AMLA_STAMP(prm, part, 19, un);
        }
        ++un;
      }
      if (!ok) report_timeout(prm.status);
    } else if (wid == 4) {
      // ---- TMA producers: V, two ring slots per page (256 columns each, one 3-D box per slot); lane l owns ring slot l
      {
        Cursor<false> cur(iter, u, have);
        int my_gv = lane;                       // next slot of the sequence this lane loads (page = gv / 2)
        uint32_t par = 1;
        bool fin = lane >= kNumVSlots, have = false;
        int page = 0;
        int issued = 0;
        const uint32_t my_full = bar(B_VFULL + lane), my_empty = bar(B_VEMPTY + lane);
        const uint32_t dst = smem_base + kOffV + lane * kVSlotBytes;
        uint64_t t_start = global_timer_ns();     // restarted whenever a lane issues a load
        bool progress = false;
        for (uint32_t spin = 0;; ++spin) {
          if (!fin && !have) {
            int lt;
            if (cur.locate(my_gv >> 1, lt)) {
              const int32_t* bt = prm.block_table + static_cast<size_t>(cur.u.b) * prm.max_blocks_per_seq;
              page = __ldg(bt + cur.u.t0 + lt);
              prefetch_l1(bt + min(cur.u.t0 + lt + 32, cur.u.t1 - 1));
              have = true;
            } else {
              fin = true;
            }
          }
          if (have && mbar_probe(my_empty, par)) {
            if ((my_gv & 1) == 0) AMLA_STAMP2(prm, part, 12, my_gv >> 1);
            mbar_arrive_expect_tx(my_full, kVSlotBytes);
            tma_load_3d(dst, &v_map, 0, page * kPage, (my_gv & 1) * 4, my_full);
            my_gv += kNumVSlots;
            par ^= 1;
            ++issued;
            have = false;
            progress = true;
          }
          if (__all_sync(0xffffffffu, fin)) break;
          // nothing to issue right now: back off, so that the polling does not take issue slots from the warps that
          // share this scheduler
          if (__any_sync(0xffffffffu, progress)) t_start = global_timer_ns(); else __nanosleep(100);
          progress = false;
          if ((spin & 1023u) == 1023u && __any_sync(0xffffffffu, global_timer_ns() - t_start > kWaitLimitNs)) { ok = false; break; }
        }
        if (!ok) {
          if (lane == 0) report_timeout(prm.status);
          if (issued > 0 && lane < kNumVSlots) mbar_wait(my_full, (issued - 1) & 1);
        }
      }
    } else if (wid == 5) {
      // ---- MMA issuer: O (+)= P~ V_t ; two N = 256 halves, four K = 16 steps each
      if (lane == 0) {
        constexpr uint32_t idesc = make_idesc_bf16(128, 256, false, true);
        constexpr uint32_t dhi = smem_desc_hi_sw128(1024);
        const uint32_t vlo0 = smem_desc_lo(smem_base + kOffV, kBoxBytes);
        const uint32_t plo0 = smem_desc_lo(smem_base + kOffP, 16);
        uint32_t slot = 0, vpar = 0;
        for (; ok && have; have = iter.next(u)) {
          for (int t = u.t0; t < u.t1 && ok; ++t, ++gt) {
            const uint32_t s = gt % kNumP, k = gt / kNumP;
            ok = mbar_wait<true>(bar(B_PFULL + s), k & 1);
            if (!ok) break;
            ok = mbar_wait(bar(B_OREADY + s), k & 1);
            if (!ok) break;
            tc_fence_after_sync();         // the correction warps may have rewritten O (tcgen05.st) before arriving
            fence_proxy_async_smem();      // P~ was written through the generic proxy (remote asynchronous stores)
            const uint32_t plo = plo0 + s * (kPStride >> 4);
            const uint32_t acc0 = t > u.t0 ? 1u : 0u;
#pragma unroll 1
            for (int nh = 0; nh < 2; ++nh) {
              ok = mbar_wait(bar(B_VFULL) + 8 * slot, vpar);
              if (!ok) break;
              if (nh == 0) AMLA_STAMP2(prm, part, 15, gt);
              uint32_t vlo = vlo0 + slot * (kVSlotBytes >> 4);
              uint32_t pl = plo;
              uint32_t acc = acc0;
#pragma unroll
              for (int kk = 0; kk < 4; ++kk)
                mma_ss(tbase + nh * 256, smem_desc_join(pl + 2 * kk, dhi), smem_desc_join(vlo + 128 * kk, dhi), idesc, kk == 0 ? acc : 1u);
              mma_commit(bar(B_VEMPTY) + 8 * slot);
              if (++slot == kNumVSlots) { slot = 0; vpar ^= 1; }
            }
            if (!ok) break;
            mma_commit_multicast(bar(X_PV + s), 3);   // PVDONE here, PEMPTY in the score CTA
            AMLA_STAMP(prm, part, 16, gt);
          }
          if (!ok) break;
        }
        if (!ok) report_timeout(prm.status);
      }
    }
  }

  // teardown: nobody may still be writing into a peer that has exited
  tc_fence_before_sync();
  __syncthreads();
  if (tid == 0) AMLA_STAMP_NS(prm, part, is_score ? 90 : 94);        // roles done
  cluster_arrive();
  cluster_wait();
  if (wid == 5) tmem_dealloc(tbase, kTmemCols);
  if (tid == 0) AMLA_STAMP_NS(prm, part, is_score ? 91 : 95);        // exit
}

// ---------------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------------
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

template <int kMode, bool kGuard>
cudaError_t launch_variant(const CUtensorMap& map, const CUtensorMap& vmap, const CUtensorMap& qmap, const DecodeParams& prm, cudaStream_t stream) {
  auto kern = decode_tc_kernel<kMode, kGuard>;
  // the opt-in to large dynamic shared memory is per device and per kernel; do it once each
  static std::atomic<uint64_t> done{0};
  int device = 0;
  cudaError_t err = cudaGetDevice(&device);
  if (err != cudaSuccess) return err;
  const uint64_t bit = 1ull << (device & 63);
  if (!(done.load(std::memory_order_acquire) & bit)) {
    err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kSmemBytes));
    if (err != cudaSuccess) return err;
    done.fetch_or(bit, std::memory_order_release);
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2 * prm.P);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kern, map, vmap, qmap, prm);
}

}  // namespace

// Number of two-CTA clusters the schedule is cut into: one per SM pair.
int decode_tc_parts(int sm_count) { return sm_count / 2 > 0 ? sm_count / 2 : 1; }

cudaError_t launch_decode_tc(const DecodeParams& prm, cudaStream_t stream, int* unsupported) {
  *unsupported = 0;
  EncodeTiledFn encode = get_encode_fn();
  if (!encode) { *unsupported = 1; return cudaErrorNotSupported; }
  // K: the cache seen as (64 columns, 8 rows of a group, 9 column blocks, row groups); one box = a page's 64 keys x
  // 3 column blocks, laid out in shared memory as [row group][column block][8 keys][64 columns], so that a
  // K-major operand descriptor with a group stride of 3 KB walks the keys of one column block.
  CUtensorMap map;
  const cuuint64_t dims[4] = {64, 8, static_cast<cuuint64_t>(kDqk / 64), static_cast<cuuint64_t>(prm.num_blocks) * 8};
  const cuuint64_t strides[3] = {static_cast<cuuint64_t>(kDqk) * 2, 128, static_cast<cuuint64_t>(kDqk) * 2 * 8};
  const cuuint32_t box[4] = {64, 8, 3, 8};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  const CUresult cr = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(prm.kv), dims, strides,
                             box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  // V: the same rows seen as (64 columns, rows, column block); one box = 64 keys x 4 column blocks, laid out in
  // shared memory as [column block][key][64 columns] -- four of the 2-D boxes above in one instruction.
  CUtensorMap vmap;
  {
    const cuuint64_t vdims[3] = {64, static_cast<cuuint64_t>(prm.num_blocks) * kPage, static_cast<cuuint64_t>(kDqk / 64)};
    const cuuint64_t vstrides[2] = {static_cast<cuuint64_t>(kDqk) * 2, 128};
    const cuuint32_t vbox[3] = {64, 64, 4};
    const cuuint32_t vestr[3] = {1, 1, 1};
    const CUresult vr = encode(&vmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(prm.kv), vdims, vstrides,
                               vbox, vestr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (vr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  // Q: (64 columns, rows of all sequences, 9 column blocks); one box = a unit's 128 rows x one column block, laid out
  // [row][64 columns] like an operand tile.  Rows past the end of the array read as zero; rows of a following
  // sequence that a short unit's box covers are dropped by the kernel.
  CUtensorMap qmap;
  {
    const cuuint64_t qdims[3] = {64, static_cast<cuuint64_t>(prm.B) * prm.R, static_cast<cuuint64_t>(kDqk / 64)};
    const cuuint64_t qstrides[2] = {static_cast<cuuint64_t>(kDqk) * 2, 128};
    const cuuint32_t qbox[3] = {64, kRowBlock, 1};
    const cuuint32_t qestr[3] = {1, 1, 1};
    const CUresult qr = encode(&qmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(prm.q), qdims, qstrides,
                               qbox, qestr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (qr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  }
  const int mode = prm.flags & 3;
  const bool guard = !(prm.flags & 4);
  if (mode == 0) return guard ? launch_variant<0, true>(map, vmap, qmap, prm, stream) : launch_variant<0, false>(map, vmap, qmap, prm, stream);
  if (mode == 1) return guard ? launch_variant<1, true>(map, vmap, qmap, prm, stream) : launch_variant<1, false>(map, vmap, qmap, prm, stream);
  return launch_variant<2, true>(map, vmap, qmap, prm, stream);
}

}  // namespace amla

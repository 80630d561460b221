// Scalar (CUDA-core) bring-up kernel for paged MLA decode with Algorithm 2's rescaling.
// It follows the same split-KV schedule, state recurrence and output conventions as the
// tensor-core kernel, one warp per query row, and exists to validate those pieces; it is only
// reachable through AMLA_FLAG_KERNEL_SIMT and is never chosen automatically.
#include "amla_common.cuh"

namespace amla {

namespace {
constexpr int kWarps = 8;
constexpr int kRowsPerWarp = 2;
constexpr int kRowsPerPass = kWarps * kRowsPerWarp;   // 16
constexpr int kKStrideW = 289;                        // words per K row in smem (578 bf16): odd => conflict-free
constexpr int kQStrideW = 288;
}  // namespace

template <int kMode, bool kGuard>
__global__ void __launch_bounds__(kWarps * 32) decode_simt_kernel(DecodeParams prm) {
  extern __shared__ uint32_t smem[];
  uint32_t* Ksm = smem;                                   // [64][289] words (bf16x2)
  uint32_t* Qsm = smem + kPage * kKStrideW;               // [16][288] words

  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5;
  const Plan plan = Plan::make(prm.prefix, prm.n_items, prm.P, prm.ovh);
  if (plan.L <= 0) return;
  const int p = blockIdx.x;
  if (p >= plan.P) return;
  const int g0 = plan.part_start(p), g1 = plan.part_start(p + 1);

  int g = g0;
  while (g < g1) {
    const int it = plan.item_of_tile(g);
    const int a = plan.first_tile(it), e = prm.prefix[it + 1];
    const int lo = max(g, a), hi = min(e, g1);
    g = min(e, g1);
    if (hi <= lo) continue;                  // only overhead positions of this item fell into the part
    const int t0 = lo - a, t1 = hi - a;
    const int b = it / prm.nrb, rb = it % prm.nrb;
    const int r0 = rb * kRowBlock;
    const int nrows = min(kRowBlock, prm.R - r0);
    const int n_b = min(max(prm.seqlens[b], 0), prm.max_blocks_per_seq * kPage);
    int p_first, p_last;
    const int nsplit = plan.item_parts(it, &p_first, &p_last);
    const int slot = nsplit == 1 ? -1 : plan.slot_of(p, it, p_first);
    if (tid == 0) prm.item_info[it] = make_int2(plan.slot_of(p_first, it, p_first), nsplit);
    const int32_t* bt = prm.block_table + static_cast<size_t>(b) * prm.max_blocks_per_seq;

    for (int pass = 0; pass * kRowsPerPass < nrows; ++pass) {
      __syncthreads();
      // stage this pass's 16 query rows (zeros beyond the last valid row)
      for (int i = tid; i < kRowsPerPass * kQStrideW; i += blockDim.x) {
        const int rl = i / kQStrideW, w = i % kQStrideW;
        const int row = pass * kRowsPerPass + rl;
        uint32_t v = 0;
        if (row < nrows)
          v = reinterpret_cast<const uint32_t*>(prm.q + (static_cast<size_t>(b) * prm.R + r0 + row) * kDqk)[w];
        Qsm[i] = v;
      }
      RowState st[kRowsPerWarp];
      float O[kRowsPerWarp][16];
#pragma unroll
      for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        row_state_init(st[rr]);
#pragma unroll
        for (int i = 0; i < 16; ++i) O[rr][i] = 0.f;
      }

      for (int t = t0; t < t1; ++t) {
        __syncthreads();
        const int page = bt[t];
        const uint32_t* src = reinterpret_cast<const uint32_t*>(prm.kv + static_cast<size_t>(page) * kPage * kDqk);
        for (int i = tid; i < kPage * kQStrideW; i += blockDim.x) {
          const int j = i / kQStrideW, w = i % kQStrideW;
          Ksm[j * kKStrideW + w] = src[i];
        }
        __syncthreads();
#pragma unroll
        for (int rr = 0; rr < kRowsPerWarp; ++rr) {
          const int rl = wid * kRowsPerWarp + rr;
          const int row = pass * kRowsPerPass + rl;
          if (row >= nrows) continue;
          const int tok = (r0 + row) / prm.H;
          const int visible = min(n_b, n_b - prm.Sq + tok + 1);
          // C1: two keys per lane
          float acc0 = 0.f, acc1 = 0.f;
          const uint32_t* qr = Qsm + rl * kQStrideW;
          const uint32_t* k0 = Ksm + lane * kKStrideW;
          const uint32_t* k1 = Ksm + (lane + 32) * kKStrideW;
#pragma unroll 8
          for (int w = 0; w < kQStrideW; ++w) {
            const float2 qf = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(qr + w));
            const float2 ka = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(k0 + w));
            const float2 kb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(k1 + w));
            acc0 = fmaf(qf.x, ka.x, acc0); acc0 = fmaf(qf.y, ka.y, acc0);
            acc1 = fmaf(qf.x, kb.x, acc1); acc1 = fmaf(qf.y, kb.y, acc1);
          }
          const int j0 = t * kPage + lane, j1 = j0 + 32;
          const float a0 = j0 < visible ? acc0 * prm.scale_log2 : -INFINITY;
          const float a1 = j1 < visible ? acc1 * prm.scale_log2 : -INFINITY;
          float tmax = fmaxf(a0, a1);
#pragma unroll
          for (int o = 16; o; o >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, o));
          // V1: scalar recurrence + probabilities
          const RowStep sp = row_step<kMode>(st[rr], tmax, prm.tau);
          const float p0 = ex2_approx(a0 - sp.m2_sub), p1 = ex2_approx(a1 - sp.m2_sub);
          float rs = p0 + p1;
#pragma unroll
          for (int o = 16; o; o >>= 1) rs += __shfl_xor_sync(0xffffffffu, rs, o);
          st[rr].l = st[rr].l * sp.l_up + rs;
          const float pt0 = bf16_round(p0 * sp.p_scale), pt1 = bf16_round(p1 * sp.p_scale);
          // rescale of the accumulator row
          if (kMode == 2) {
            if (sp.l_up != 1.f) {
#pragma unroll
              for (int i = 0; i < 16; ++i) O[rr][i] *= sp.l_up;
            }
          } else if (sp.n_bits != 0) {
#pragma unroll
            for (int i = 0; i < 16; ++i)
              O[rr][i] = kGuard ? exponent_add_guarded(O[rr][i], sp.n_bits) : exponent_add_raw(O[rr][i], sp.n_bits);
          }
          // C2: O += P~ V
#pragma unroll 4
          for (int j = 0; j < kPage; ++j) {
            const float pj = __shfl_sync(0xffffffffu, j < 32 ? pt0 : pt1, j & 31);
            const uint32_t* vr = Ksm + j * kKStrideW + lane;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(vr + 32 * i));
              O[rr][2 * i] = fmaf(pj, v.x, O[rr][2 * i]);
              O[rr][2 * i + 1] = fmaf(pj, v.y, O[rr][2 * i + 1]);
            }
          }
        }
      }
      // finalise: O / (l * S16); lse = m + ln l
#pragma unroll
      for (int rr = 0; rr < kRowsPerWarp; ++rr) {
        const int row = pass * kRowsPerPass + wid * kRowsPerWarp + rr;
        if (row >= nrows) continue;
        const bool live = st[rr].l > 0.f;
        const float inv = live ? prm.out_scale / (st[rr].l * st[rr].s_out) : 0.f;
        const float lse = live ? (st[rr].m2 + log2f(st[rr].l)) * kLn2 : -INFINITY;
        if (slot < 0) {
          __nv_bfloat16* orow = prm.out + (static_cast<size_t>(b) * prm.R + r0 + row) * kDv;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            __nv_bfloat162 v = __floats2bfloat162_rn(O[rr][2 * i] * inv, O[rr][2 * i + 1] * inv);
            reinterpret_cast<__nv_bfloat162*>(orow)[lane + 32 * i] = v;
          }
          if (lane == 0) prm.lse[static_cast<size_t>(b) * prm.R + r0 + row] = lse;
        } else {
          // half precision with one power-of-two scale per 32-column chunk (see "Split partials"): the 16 lanes of a
          // half-warp hold one chunk of the row in every round
          const size_t prow = static_cast<size_t>(slot) * kRowBlock + row;
          uint32_t* hrow = reinterpret_cast<uint32_t*>(partial_halves(prm) + prow * kDv);
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const float x0 = O[rr][2 * i] * inv, x1 = O[rr][2 * i + 1] * inv;
            float mx = fmaxf(fabsf(x0), fabsf(x1));
#pragma unroll
            for (int o = 8; o; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            float f;
            const uint32_t sb = partial_scale_byte(mx, &f);
            hrow[lane + 32 * i] = pack_f16x2(x0 * f, x1 * f);
            if ((lane & 15) == 0) partial_scales(prm)[prow * 16 + 2 * i + (lane >> 4)] = static_cast<uint8_t>(sb);
          }
          if (lane == 0) prm.part_lse[prow] = lse;
        }
      }
    }
  }
}

cudaError_t launch_decode_simt(const DecodeParams& prm, cudaStream_t stream) {
  const size_t smem = (kPage * kKStrideW + kRowsPerPass * kQStrideW) * sizeof(uint32_t);
  const int mode = prm.flags & 3;
  const bool guard = !(prm.flags & 4);
  void (*kern)(DecodeParams) = nullptr;
  if (mode == 0) kern = guard ? decode_simt_kernel<0, true> : decode_simt_kernel<0, false>;
  else if (mode == 1) kern = guard ? decode_simt_kernel<1, true> : decode_simt_kernel<1, false>;
  else kern = decode_simt_kernel<2, true>;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) return err;
  kern<<<prm.P, kWarps * 32, smem, stream>>>(prm);
  return cudaGetLastError();
}

}  // namespace amla

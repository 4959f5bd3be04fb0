// Self-attention with log2-quantized scores (Sec. 3.3, Eq. 2) on the tcgen05 tensor cores.
//
//     A = softmax(Q K^T / sqrt(d)),  code = clamp(rint(-log2(A / s)), 0, 2^b - 1),  O = s sum_j 2^-code_j V_j
//
// One CTA owns 128 query rows of one (prompt, head) and walks the keys in blocks of 128 two or three
// times:
//   walk "max"   : S = Q K^T into tensor memory, every row keeps its largest logit;
//   walk "sum"   : (fixed scale only) the row sums of 2^(t - max), which the codes then depend on;
//   walk "codes" : S again; code = rint(base - t) in the log domain, P = 2^(14 - code) as fp16 into a
//                  shared-memory operand tile, O += P V on the tensor cores.  With the row maximum as
//                  scale the codes do not depend on the row sum, which is then gathered in this walk.
// Roles: 16 softmax warps (warp w reads tensor-memory lanes 32 (w % 4) .. +31, columns 32 (w / 4) .. +31
// of every score block), one TMA producer lane, one MMA issuer lane.  Q, K and P are K-major operands
// with 128-byte swizzled rows; V is used as it lies in memory (features contiguous), an MN-major operand.
// Tiles are fetched as boxes of 64 features x 128 tokens; features beyond d and tokens beyond the
// sequence are zero-filled by the copy engine, so d = 40 runs as 48 and ragged ends need no staging.
#pragma once

#include "self_attention.cuh"

namespace dgq {

constexpr int SATC_SOFTMAX_WARPS = 16;
constexpr int SATC_WARP_TMA = 16;
constexpr int SATC_WARP_MMA = 17;
constexpr int SATC_THREADS = 18 * 32;
constexpr int SATC_BQ = 128;            // query rows per CTA
constexpr int SATC_BK = 128;            // keys per block
constexpr int SATC_PANEL = 128 * 128;   // bytes of one 64-feature (or 64-key) panel of 128 rows
constexpr int SATC_TMEM_O = 256;        // column of the output accumulator (score buffers at 0 and 128)

template <int D>
struct SaTcCfg {
  static constexpr int DP = (D + 15) / 16 * 16;
  static constexpr int NP = (D + 63) / 64;
  static constexpr int KSTEPS = DP / 16;
  static constexpr int KST = NP == 1 ? 3 : (NP == 2 ? 2 : 1);
  static constexpr int VST = NP == 1 ? 2 : 1;
  static constexpr int PST = NP <= 2 ? 2 : 1;
  static constexpr int TILE = NP * SATC_PANEL;
  static constexpr int P_TILE = 2 * SATC_PANEL;
  static constexpr int OFF_K = TILE;
  static constexpr int OFF_V = OFF_K + KST * TILE;
  static constexpr int OFF_P = OFF_V + VST * TILE;
  static constexpr int OFF_SH = OFF_P + PST * P_TILE;
  static constexpr int SMEM = 1024 + OFF_SH + 1024 + 2 * 4 * SATC_BQ * 4;
  static_assert(SMEM <= 232448, "shared memory budget");
};

struct SaTcShared {
  uint64_t q_full;
  uint64_t k_full[3], k_empty[3];
  uint64_t v_full[2], v_empty[2];
  uint64_t s_full[2], s_free[2];
  uint64_t p_full[2], p_free[2];
  uint64_t o_full;
  uint32_t tmem_base;
  int abort_flag;
};

__device__ __forceinline__ void mma_f16(uint32_t d_tmem, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                        uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// MN-major operand with 128-byte swizzled rows (one row = 64 contiguous elements of the M/N axis for
// one k): `lbo` = bytes between 64-element blocks of the M/N axis, `sbo` = bytes between groups of 8 k.
__device__ __forceinline__ uint64_t smem_desc_mn(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  return (uint64_t)((addr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo_bytes >> 4) << 16) | ((uint64_t)(sbo_bytes >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
__device__ __forceinline__ void named_bar_sync(int id, int n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

// kind::f16 instruction descriptor: fp32 accumulator (bits 4-5 = 1), fp16 A and B (format 0), B major at
// bit 16 (1 = MN-major), N >> 3 at bit 17, M >> 4 at bit 24.
__host__ __device__ constexpr uint32_t satc_idesc(int n, bool b_mn_major) {
  return (1u << 4) | ((b_mn_major ? 1u : 0u) << 16) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(SATC_BQ >> 4) << 24);
}

template <int D, bool FIXED, bool CODES>
__global__ void __launch_bounds__(SATC_THREADS, 1)
self_attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                    const __grid_constant__ CUtensorMap tmV, const __grid_constant__ SelfAttnArgs a) {
  using Cfg = SaTcCfg<D>;
  constexpr int NP = Cfg::NP, KST = Cfg::KST, VST = Cfg::VST, PST = Cfg::PST;
  constexpr int N_WALKS = FIXED ? 3 : 2;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                         ~uintptr_t(1023));
  unsigned char* sQ = smem;
  unsigned char* sK = smem + Cfg::OFF_K;
  unsigned char* sV = smem + Cfg::OFF_V;
  unsigned char* sP = smem + Cfg::OFF_P;
  SaTcShared* sh = reinterpret_cast<SaTcShared*>(smem + Cfg::OFF_SH);
  float* mpart = reinterpret_cast<float*>(smem + Cfg::OFF_SH + 1024);  // [4][128] partial row maxima
  float* zpart = mpart + 4 * SATC_BQ;                                  // [4][128] partial row sums
  volatile int* abort_flag = &sh->abort_flag;

  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  const int row0 = rb * SATC_BQ;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nb = (a.nk + SATC_BK - 1) / SATC_BK;

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    mbar_init(&sh->q_full, 1);
    for (int i = 0; i < 3; ++i) {
      mbar_init(&sh->k_full[i], 1);
      mbar_init(&sh->k_empty[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&sh->v_full[i], 1);
      mbar_init(&sh->v_empty[i], 1);
      mbar_init(&sh->s_full[i], 1);
      mbar_init(&sh->s_free[i], SATC_SOFTMAX_WARPS);
      mbar_init(&sh->p_full[i], SATC_SOFTMAX_WARPS);
      mbar_init(&sh->p_free[i], 1);
    }
    mbar_init(&sh->o_full, 1);
    sh->abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == SATC_WARP_MMA) {
    tmem_alloc(&sh->tmem_base, 512);
    tmem_relinquish();
  }
  pdl_wait();  // Q, K and V may come from earlier kernels
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = sh->tmem_base;

  if (warp == SATC_WARP_TMA) {
    // ------------------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      tma_prefetch_desc(&tmQ);
      tma_prefetch_desc(&tmK);
      tma_prefetch_desc(&tmV);
      mbar_arrive_expect_tx(&sh->q_full, (uint32_t)Cfg::TILE);
      for (int p = 0; p < NP; ++p) tma_load_4d(sQ + p * SATC_PANEL, &tmQ, &sh->q_full, p * 64, h, row0, b);
      uint32_t it = 0, vit = 0;
      for (int w = 0; w < N_WALKS && !*abort_flag; ++w) {
        const bool last = (w == N_WALKS - 1);
        for (int j = 0; j < nb; ++j) {
          const uint32_t ks = it % KST;
          mbar_wait_lean(smem_u32(&sh->k_empty[ks]), ((it / KST) & 1u) ^ 1u, abort_flag);
          mbar_arrive_expect_tx(&sh->k_full[ks], (uint32_t)Cfg::TILE);
          for (int p = 0; p < NP; ++p)
            tma_load_4d(sK + ks * Cfg::TILE + p * SATC_PANEL, &tmK, &sh->k_full[ks], p * 64, h, j * SATC_BK, b);
          ++it;
          if (last) {
            const uint32_t vs = vit % VST;
            mbar_wait_lean(smem_u32(&sh->v_empty[vs]), ((vit / VST) & 1u) ^ 1u, abort_flag);
            mbar_arrive_expect_tx(&sh->v_full[vs], (uint32_t)Cfg::TILE);
            for (int p = 0; p < NP; ++p)
              tma_load_4d(sV + vs * Cfg::TILE + p * SATC_PANEL, &tmV, &sh->v_full[vs], p * 64, h, j * SATC_BK, b);
            ++vit;
          }
          if (*abort_flag) break;
        }
      }
    }
    __syncwarp();
  } else if (warp == SATC_WARP_MMA) {
    // ------------------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = satc_idesc(SATC_BK, false);
      constexpr uint32_t IDESC_PV = satc_idesc(Cfg::DP, true);
      const uint32_t q_addr = smem_u32(sQ), k_addr = smem_u32(sK), v_addr = smem_u32(sV), p_addr = smem_u32(sP);
      uint32_t it = 0, pit = 0;
      // O += P V of the block whose P tile is `pit` in ring order
      auto issue_pv = [&](int jj) {
        const uint32_t pb = pit % PST, vs = pit % VST;
        mbar_wait_lean(smem_u32(&sh->p_full[pb]), (pit / PST) & 1u, abort_flag);
        mbar_wait_lean(smem_u32(&sh->v_full[vs]), (pit / VST) & 1u, abort_flag);
        tc_fence_after();
#pragma unroll
        for (int kstep = 0; kstep < SATC_BK / 16; ++kstep) {
          const uint64_t da = smem_desc(p_addr + pb * Cfg::P_TILE + (kstep >> 2) * SATC_PANEL + (kstep & 3) * 32, 1024, 2);
          const uint64_t db = smem_desc_mn(v_addr + vs * Cfg::TILE + kstep * 2048, SATC_PANEL, 1024);
          mma_f16(tmem_base + SATC_TMEM_O, da, db, IDESC_PV, (jj > 0 || kstep > 0) ? 1u : 0u);
        }
        mma_commit(&sh->v_empty[vs]);
        mma_commit(&sh->p_free[pb]);
        ++pit;
      };
      mbar_wait_lean(smem_u32(&sh->q_full), 0, abort_flag);
      for (int w = 0; w < N_WALKS && !*abort_flag; ++w) {
        const bool last = (w == N_WALKS - 1);
        for (int j = 0; j < nb; ++j) {
          const uint32_t ks = it % KST, sb = it & 1u;
          mbar_wait_lean(smem_u32(&sh->k_full[ks]), (it / KST) & 1u, abort_flag);
          mbar_wait_lean(smem_u32(&sh->s_free[sb]), ((it >> 1) & 1u) ^ 1u, abort_flag);
          tc_fence_after();
#pragma unroll
          for (int kstep = 0; kstep < Cfg::KSTEPS; ++kstep) {
            const uint32_t off = (kstep >> 2) * SATC_PANEL + (kstep & 3) * 32;
            mma_f16(tmem_base + sb * SATC_BK, smem_desc(q_addr + off, 1024, 2),
                    smem_desc(k_addr + ks * Cfg::TILE + off, 1024, 2), IDESC_QK, kstep > 0 ? 1u : 0u);
          }
          mma_commit(&sh->k_empty[ks]);
          mma_commit(&sh->s_full[sb]);
          ++it;
          if (last && j > 0) issue_pv(j - 1);  // after the next block's scores, so the softmax warps stay fed
          if (*abort_flag) break;
        }
        if (last && !*abort_flag) {
          issue_pv(nb - 1);
          mma_commit(&sh->o_full);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax / quantizer warps
    const int q = warp & 3, cp = warp >> 2;
    const int row = q * 32 + lane;                       // row of the CTA's tile
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    const float scale = a.qk_scale_log2;
    const float Lf = (float)((1 << a.bits) - 1);
    const float Lclamp = CODES ? Lf : fminf(Lf, AT_CODE_CAP);
    uint32_t it = 0, pit = 0;
    float m_raw = -INFINITY, m2 = 0.f, base = 0.f, zsum = 0.f;
    for (int w = 0; w < N_WALKS; ++w) {
      const bool walk_max = (w == 0), walk_codes = (w == N_WALKS - 1);
      for (int j = 0; j < nb; ++j) {
        const uint32_t sb = it & 1u;
        // After a time-out every wait returns at once and the loops run to their ends on whatever the
        // buffers hold (an error is recorded): no warp leaves early, so the named barriers below are
        // always reached by all 16 warps.
        mbar_wait_lean(smem_u32(&sh->s_full[sb]), (it >> 1) & 1u, abort_flag);
        __syncwarp();
        tc_fence_after();
        uint32_t r[32];
        {
          uint32_t r0[16], r1[16];
          tmem_ld16(t_lane + sb * SATC_BK + cp * 32, r0);
          tmem_ld16(t_lane + sb * SATC_BK + cp * 32 + 16, r1);
          tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            r[i] = r0[i];
            r[16 + i] = r1[i];
          }
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&sh->s_free[sb]);
        ++it;
        const int valid = a.nk - j * SATC_BK - cp * 32;  // this warp's columns below `valid` are real keys
        if (valid < 32) {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (i >= valid) r[i] = 0xFF800000u;  // -inf
        }
        if (walk_max) {
#pragma unroll
          for (int i = 0; i < 32; ++i) m_raw = fmaxf(m_raw, __uint_as_float(r[i]));
        } else if (!walk_codes) {
          // row sums with the final maximum (fixed scale: the codes need them first)
#pragma unroll
          for (int i = 0; i < 32; ++i) zsum += ex2_approx(fmaf(__uint_as_float(r[i]), scale, -m2));
        } else {
          uint32_t pk[16];
          const int64_t code_row = (((int64_t)b * a.H + h) * a.nq + row0 + row) * a.nk + j * SATC_BK + cp * 32;
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            float pf[2];
#pragma unroll
            for (int e = 0; e < 2; ++e) {
              const float t = __uint_as_float(r[i + e]);
              if (!FIXED) zsum += ex2_approx(fmaf(t, scale, -m2));
              // rint by adding 1.5 * 2^23: the low bits of the sum are the integer; -inf logits (keys
              // beyond nk) clamp to the last code, their V rows are zero
              const float x = fminf(fmaxf(fmaf(t, -scale, base), 0.f), Lclamp);
              const uint32_t bits = __float_as_uint(x + 12582912.0f);
              if (CODES) {
                r[i + e] = bits & 0xFFu;
                const uint32_t capped = min(bits, 0x4B400000u + (uint32_t)AT_CODE_CAP);
                pf[e] = __uint_as_float(0x46800000u - (capped << 23));
              } else {
                pf[e] = __uint_as_float(0x46800000u - (bits << 23));  // 2^(14 - code)
              }
            }
            const __half2 ph = __floats2half2_rn(pf[0], pf[1]);
            pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&ph);
          }
          if (CODES && row0 + row < a.nq) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i < valid) a.codes_out[code_row + i] = (uint8_t)r[i];
          }
          const uint32_t pb = pit % PST;
          mbar_wait_lean(smem_u32(&sh->p_free[pb]), ((pit / PST) & 1u) ^ 1u, abort_flag);
          __syncwarp();
          unsigned char* prow = sP + pb * Cfg::P_TILE + (cp >> 1) * SATC_PANEL + row * 128;
#pragma unroll
          for (int c = 0; c < 4; ++c)
            *reinterpret_cast<uint4*>(prow + ((((cp & 1) * 4 + c) ^ (row & 7)) << 4)) =
                make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
          fence_proxy_async_smem();
          __syncwarp();
          if (lane == 0) mbar_arrive(&sh->p_full[pb]);
          ++pit;
        }
      }
      if (walk_max) {
        mpart[cp * SATC_BQ + row] = m_raw;
        named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
        m_raw = fmaxf(fmaxf(mpart[row], mpart[SATC_BQ + row]), fmaxf(mpart[2 * SATC_BQ + row], mpart[3 * SATC_BQ + row]));
        m2 = m_raw * scale;
        base = m2;  // row maximum as scale: log2 s + max + log2 sum = max
      } else if (!walk_codes) {
        zpart[cp * SATC_BQ + row] = zsum;
        named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
        zsum = (zpart[row] + zpart[SATC_BQ + row]) + (zpart[2 * SATC_BQ + row] + zpart[3 * SATC_BQ + row]);
        const float log2_fixed = log2f(fmaxf(__ldg(a.fixed_scale + b), 1.17549435e-38f));
        base = log2_fixed + m2 + log2f(zsum);
      }
    }
    {
      float s_row;
      if (FIXED) {
        s_row = fmaxf(__ldg(a.fixed_scale + b), 1.17549435e-38f);
      } else {
        zpart[cp * SATC_BQ + row] = zsum;
        named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
        s_row = 1.0f / ((zpart[row] + zpart[SATC_BQ + row]) + (zpart[2 * SATC_BQ + row] + zpart[3 * SATC_BQ + row]));
      }
      s_row *= 6.103515625e-05f;  // 2^-14
      mbar_wait_lean(smem_u32(&sh->o_full), 0, abort_flag);
      __syncwarp();
      {
        tc_fence_after();
        __half* o_row = a.O + (((int64_t)b * a.nq + row0 + row) * a.H + h) * D;
        for (int ch = cp; ch < D / 8; ch += 4) {
          uint32_t o[8];
          tmem_ld8(t_lane + SATC_TMEM_O + ch * 8, o);
          tmem_ld_wait();
          __half2 oh[4];
#pragma unroll
          for (int i = 0; i < 4; ++i)
            oh[i] = __floats2half2_rn(s_row * __uint_as_float(o[2 * i]), s_row * __uint_as_float(o[2 * i + 1]));
          if (row0 + row < a.nq) *(reinterpret_cast<uint4*>(o_row) + ch) = *reinterpret_cast<const uint4*>(oh);
        }
      }
    }
  }

  // ------------------------------------------------------------ common exit
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the CTA's shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 200000) {
    }
    __syncthreads();
  }
  if (warp == SATC_WARP_MMA) {
    __syncwarp();
    tc_fence_after();
    tmem_dealloc(tmem_base, 512);
  }
}

// [B, n, H, d] fp16 as a 4-D tensor (d, H, n, B); boxes of 64 features x 128 tokens of one head.
static bool satc_encode(CUtensorMap* m, const void* base, int B, int n, int H, int d) {
  const uint64_t dims[4] = {(uint64_t)d, (uint64_t)H, (uint64_t)n, (uint64_t)B};
  const uint64_t strides[3] = {(uint64_t)d * 2, (uint64_t)H * d * 2, (uint64_t)n * H * d * 2};
  const uint32_t box[4] = {64, 1, 128, 1};
  return encode_map(m, base, 4, dims, strides, box, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_DATA_TYPE_FLOAT16);
}

template <int D, bool FIXED, bool CODES>
static dgq_status launch_self_attn_tc2(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                       const SelfAttnArgs& a, unsigned grid, cudaStream_t stream) {
  using Cfg = SaTcCfg<D>;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(self_attn_tc_kernel<D, FIXED, CODES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg::SMEM));
    if (dev < 64) attr_set[dev] = true;
  }
  DGQ_CUDA_OK(launch_pdl(self_attn_tc_kernel<D, FIXED, CODES>, dim3(grid), dim3(SATC_THREADS), (size_t)Cfg::SMEM, stream,
                         tmQ, tmK, tmV, a));
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

template <int D>
static dgq_status launch_self_attn_tc(const SelfAttnArgs& a, cudaStream_t stream) {
  SelfAttnArgs aa = a;
  aa.n_row_blocks = (a.nq + SATC_BQ - 1) / SATC_BQ;
  const int64_t grid = (int64_t)a.B * a.H * aa.n_row_blocks;
  if (grid > INT_MAX) return DGQ_ERR_UNSUPPORTED;
  CUtensorMap tmQ, tmK, tmV;
  std::memset(&tmQ, 0, sizeof(tmQ));
  std::memset(&tmK, 0, sizeof(tmK));
  std::memset(&tmV, 0, sizeof(tmV));
  if (!satc_encode(&tmQ, a.Q, a.B, a.nq, a.H, D) || !satc_encode(&tmK, a.K, a.B, a.nk, a.H, D) ||
      !satc_encode(&tmV, a.V, a.B, a.nk, a.H, D))
    return DGQ_ERR_CUDA;
  const unsigned g = (unsigned)grid;
  if (a.fixed_scale)
    return a.codes_out ? launch_self_attn_tc2<D, true, true>(tmQ, tmK, tmV, aa, g, stream)
                       : launch_self_attn_tc2<D, true, false>(tmQ, tmK, tmV, aa, g, stream);
  return a.codes_out ? launch_self_attn_tc2<D, false, true>(tmQ, tmK, tmV, aa, g, stream)
                     : launch_self_attn_tc2<D, false, false>(tmQ, tmK, tmV, aa, g, stream);
}

}  // namespace dgq

extern "C" dgq_status dgq_self_attn_logq(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk,
                                         int d, int score_bits, const float* fixed_scale, void* O,
                                         uint8_t* codes_out, void* stream) {
  using namespace dgq;
  if (!Q || !K || !V || !O || B <= 0 || H <= 0 || nq <= 0 || nk <= 0 || d <= 0) return DGQ_ERR_INVALID_ARG;
  if (score_bits < 2 || score_bits > 8) return DGQ_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return DGQ_ERR_ALIGNMENT;
  if (d != 40 && d != 64 && d != 80 && d != 128 && d != 160) return DGQ_ERR_UNSUPPORTED;
  SelfAttnArgs a;
  a.Q = (const __half*)Q;
  a.K = (const __half*)K;
  a.V = (const __half*)V;
  a.O = (__half*)O;
  a.B = B;
  a.H = H;
  a.nq = nq;
  a.nk = nk;
  a.bits = score_bits;
  a.qk_scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)d));
  a.fixed_scale = fixed_scale;
  a.codes_out = codes_out;
  a.n_row_blocks = 0;
  cudaStream_t st = (cudaStream_t)stream;
  static const bool warp_mma = [] {
    const char* e = std::getenv("DGQ_SELF_ATTN_WARP_MMA");
    return e && e[0] == '1';
  }();
  if (!warp_mma) {
    switch (d) {
      case 40: return launch_self_attn_tc<40>(a, st);
      case 64: return launch_self_attn_tc<64>(a, st);
      case 80: return launch_self_attn_tc<80>(a, st);
      case 128: return launch_self_attn_tc<128>(a, st);
      default: return launch_self_attn_tc<160>(a, st);
    }
  }
  switch (d) {
    case 40: return launch_self_attn<40>(a, st);
    case 64: return launch_self_attn<64>(a, st);
    case 80: return launch_self_attn<80>(a, st);
    case 128: return launch_self_attn<128>(a, st);
    default: return launch_self_attn<160>(a, st);
  }
}

// Self-attention with log2-quantized scores (Sec. 3.3 applies the log quantizer of Eq. 2 "to both self
// and cross-attentions") on the tcgen05 tensor cores:
//
//     A = softmax(Q K^T / sqrt(d)),  code = clamp(rint(-log2(A / s)), 0, 2^b - 1),  O = s sum_j 2^-code_j V_j
//
// with s the largest score of the query row, or one fixed scale per prompt; there is no <start> column.
// One CTA owns one or two tiles of 128 query rows of one (prompt, head) and walks the keys in blocks of
// 128 two or three times:
//   walk "max"   : S = Q K^T into tensor memory, every row keeps its largest logit;
//   walk "sum"   : (fixed scale only) the row sums of 2^(t - max), which the codes then depend on;
//   walk "codes" : S again; code = rint(base - t) in the log domain, P = 2^(14 - code) as fp16 into
//                  tensor memory, O += P V on the tensor cores with P read from there.  With the row maximum as
//                  scale the codes do not depend on the row sum, which is then gathered in this walk.
// Roles: 16 softmax warps (warp w reads tensor-memory lanes 32 (w % 4) .. +31, columns 32 (w / 4) .. +31
// of every score tile), one TMA producer lane, one lane that issues the score MMAs and one that issues
// the P V MMAs (each tile costs an issuing thread a chain of dependent instructions, so the two run apart).  With two query tiles the softmax
// warps alternate between them, so every K / V block fetched from L2 serves 256 query rows and one
// tile's MMAs run under the other tile's arithmetic.  Q, K and P are K-major operands with 128-byte
// swizzled rows; V is used as it lies in memory (features contiguous), an MN-major operand.  Tiles are
// fetched as boxes of 64 features x 128 tokens; features beyond d and tokens beyond the sequence are
// zero-filled by the copy engine, so d = 40 runs as 48 and ragged ends need no staging.
#pragma once

#include "attention.cuh"

namespace dgq {

struct SelfAttnArgs {
  const __half* Q;
  const __half* K;
  const __half* V;
  __half* O;
  int B, H, nq, nk, bits;
  float qk_scale_log2;       // log2(e) / sqrt(d)
  const float* fixed_scale;  // dev [B] or null (row maximum)
  uint8_t* codes_out;        // dev [B, H, nq, nk] or null
  int n_row_blocks;
};

constexpr int SATC_SOFTMAX_WARPS = 16;
constexpr int SATC_WARP_TMA = 16;
constexpr int SATC_WARP_MMA = 17;   // issues S = Q K^T (and owns the tensor-memory allocation)
constexpr int SATC_WARP_PV = 18;    // issues O += P V
constexpr int SATC_THREADS = 19 * 32;
constexpr int SATC_BQ = 128;            // query rows per tile
constexpr int SATC_BK = 128;            // keys per block
constexpr int SATC_PANEL = 128 * 128;   // bytes of one 64-feature (or 64-key) panel of 128 rows
constexpr int SATC_TMEM_P = 256;        // first column of the P tiles (score buffers at columns 0 and 128)

template <int D>
struct SaTcCfg {
  static constexpr int DP = (D + 15) / 16 * 16;
  static constexpr int NP = (D + 63) / 64;
  static constexpr int NT = NP == 1 ? 2 : 1;   // query tiles per CTA (shared memory and tensor memory budget)
  static constexpr int KSTEPS = DP / 16;
  static constexpr int KST = NP <= 2 ? 3 : 2;
  static constexpr int VST = NP <= 2 ? 2 : 1;
  // P = 2^(14 - code) as fp16 lives in tensor memory (64 columns per tile of 128 keys) and is the A
  // operand of P V from there: two tiles in flight where the accumulators leave room
  static constexpr int PST = (SATC_TMEM_P + 128 + NT * DP <= 512) ? 2 : 1;
  static constexpr int TMEM_O = SATC_TMEM_P + PST * 64;
  static constexpr int TILE = NP * SATC_PANEL;
  static constexpr int OFF_K = NT * TILE;
  static constexpr int OFF_V = OFF_K + KST * TILE;
  static constexpr int OFF_SH = OFF_V + VST * TILE;
  static constexpr int SMEM = 1024 + OFF_SH + 1024 + 2 * 4 * SATC_BQ * 4;
  static_assert(SMEM <= 232448, "shared memory budget");
  static_assert(TMEM_O + NT * DP <= 512, "tensor memory budget");
  static_assert(NT == 1 || PST == 2, "alternating query tiles need two P tiles");
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
// The same with the descriptors given as (low, high) words: the high words are constants of the layout,
// only the address field in the low word changes from step to step, which keeps the issuing thread's
// dependent instruction chain short (that chain, not the tensor pipe, is what bounds a tile otherwise).
__device__ __forceinline__ void mma_f16_lohi(uint32_t d_tmem, uint32_t a_lo, uint32_t a_hi, uint32_t b_lo,
                                             uint32_t b_hi, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "mov.b64 da, {%1, %2};\n\t"
      "mov.b64 db, {%3, %4};\n\t"
      "setp.ne.b32 p, %6, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(a_hi), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// A from tensor memory (128 lanes x 8 columns of packed fp16 pairs per K step of 16), B from shared memory.
__device__ __forceinline__ void mma_f16_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi,
                                           uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "setp.ne.b32 p, %5, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
      : "memory");
}
// 32 lanes x 16 consecutive 32-bit columns: thread i of the warp writes row (lane base + i).
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
        "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
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
self_attn_logq_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                      const __grid_constant__ CUtensorMap tmV, const __grid_constant__ SelfAttnArgs a) {
  using Cfg = SaTcCfg<D>;
  constexpr int NP = Cfg::NP, NT = Cfg::NT, KST = Cfg::KST, VST = Cfg::VST, PST = Cfg::PST;
  constexpr int N_WALKS = FIXED ? 3 : 2;
  extern __shared__ unsigned char smem_dyn[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_dyn) + 1023) &
                                                         ~uintptr_t(1023));
  unsigned char* sQ = smem;
  unsigned char* sK = smem + Cfg::OFF_K;
  unsigned char* sV = smem + Cfg::OFF_V;
  SaTcShared* sh = reinterpret_cast<SaTcShared*>(smem + Cfg::OFF_SH);
  float* mpart = reinterpret_cast<float*>(smem + Cfg::OFF_SH + 1024);  // [4][128] partial row maxima
  float* zpart = mpart + 4 * SATC_BQ;                                  // [4][128] partial row sums
  volatile int* abort_flag = &sh->abort_flag;

  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  const int row0 = rb * (SATC_BQ * NT);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nb = (a.nk + SATC_BK - 1) / SATC_BK;
  const int per_walk = nb * NT;  // score tiles per walk, in the order (key block, query tile)

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
      mbar_arrive_expect_tx(&sh->q_full, (uint32_t)(NT * Cfg::TILE));
      for (int t = 0; t < NT; ++t)
        for (int p = 0; p < NP; ++p)
          tma_load_4d(sQ + t * Cfg::TILE + p * SATC_PANEL, &tmQ, &sh->q_full, p * 64, h, row0 + t * SATC_BQ, b);
      uint32_t kit = 0, vit = 0;
      auto load_v = [&](int j) {
        const uint32_t vs = vit % VST;
        mbar_wait_lean(smem_u32(&sh->v_empty[vs]), ((vit / VST) & 1u) ^ 1u, abort_flag);
        mbar_arrive_expect_tx(&sh->v_full[vs], (uint32_t)Cfg::TILE);
        for (int p = 0; p < NP; ++p)
          tma_load_4d(sV + vs * Cfg::TILE + p * SATC_PANEL, &tmV, &sh->v_full[vs], p * 64, h, j * SATC_BK, b);
        ++vit;
      };
      for (int w = 0; w < N_WALKS && !*abort_flag; ++w) {
        const bool last = (w == N_WALKS - 1);
        for (int j = 0; j < nb; ++j) {
          const uint32_t ks = kit % KST;
          mbar_wait_lean(smem_u32(&sh->k_empty[ks]), ((kit / KST) & 1u) ^ 1u, abort_flag);
          mbar_arrive_expect_tx(&sh->k_full[ks], (uint32_t)Cfg::TILE);
          for (int p = 0; p < NP; ++p)
            tma_load_4d(sK + ks * Cfg::TILE + p * SATC_PANEL, &tmK, &sh->k_full[ks], p * 64, h, j * SATC_BK, b);
          ++kit;
          // V of the previous block goes out after K of this one: the scores of block j are issued
          // before P V of block j - 1, and a V stage only frees when such a product has completed
          if (last && j > 0) load_v(j - 1);
          if (*abort_flag) break;
        }
        if (last && !*abort_flag) load_v(nb - 1);
      }
    }
    __syncwarp();
  } else if (warp == SATC_WARP_MMA) {
    // ------------------------------------------------------------ score issuer (one lane)
    // Score tiles are numbered g = 0 .. N_WALKS * per_walk - 1 in the order (walk, key block, query
    // tile) and alternate between the two score buffers; a tile is issued as soon as its buffer has
    // been read, which is early in the arithmetic of tile g - 2.
    if (lane == 0) {
      constexpr uint32_t IDESC_QK = satc_idesc(SATC_BK, false);
      constexpr uint32_t HI = smem_desc_hi(1024, 2);
      const uint32_t q_lo = smem_desc_lo(smem_u32(sQ)), k_lo = smem_desc_lo(smem_u32(sK));
      const uint32_t k_full0 = smem_u32(&sh->k_full[0]), k_empty0 = smem_u32(&sh->k_empty[0]);
      const uint32_t s_full0 = smem_u32(&sh->s_full[0]), s_free0 = smem_u32(&sh->s_free[0]);
      const int total = N_WALKS * per_walk;
      uint32_t ks = 0, k_par = 0;
      mbar_wait_lean(smem_u32(&sh->q_full), 0, abort_flag);
      for (int g = 0; g < total; ++g) {
        const uint32_t sb = (uint32_t)g & 1u;
        const uint32_t t = NT == 2 ? sb : 0u;
        if (t == 0) mbar_wait_lean(k_full0 + ks * 8u, k_par, abort_flag);
        mbar_wait_lean(s_free0 + sb * 8u, (((uint32_t)g >> 1) & 1u) ^ 1u, abort_flag);
        tc_fence_after();
        const uint32_t a_lo = q_lo + t * (uint32_t)(Cfg::TILE >> 4), b_lo = k_lo + ks * (uint32_t)(Cfg::TILE >> 4);
#pragma unroll
        for (int kstep = 0; kstep < Cfg::KSTEPS; ++kstep) {
          const uint32_t off = (uint32_t)(((kstep >> 2) * SATC_PANEL + (kstep & 3) * 32) >> 4);
          mma_f16_lohi(tmem_base + sb * SATC_BK, a_lo + off, HI, b_lo + off, HI, IDESC_QK, kstep > 0 ? 1u : 0u);
        }
        if (t == NT - 1) {
          mma_commit_addr(k_empty0 + ks * 8u);
          if (++ks == (uint32_t)KST) {
            ks = 0;
            k_par ^= 1u;
          }
        }
        mma_commit_addr(s_full0 + sb * 8u);
        if ((g & 7) == 7 && *abort_flag) break;
      }
    }
    __syncwarp();
  } else if (warp == SATC_WARP_PV) {
    // ------------------------------------------------------------ product issuer (one lane)
    // O(tile) += P V for the tiles of the codes walk, each as soon as its P tile is complete.
    if (lane == 0) {
      constexpr uint32_t IDESC_PV = satc_idesc(Cfg::DP, true);
      constexpr uint32_t HI = smem_desc_hi(1024, 2);
      const uint32_t v_lo = ((smem_u32(sV) & 0x3FFFFu) >> 4) | ((uint32_t)(SATC_PANEL >> 4) << 16);  // MN-major: block stride
      const uint32_t p_full0 = smem_u32(&sh->p_full[0]), p_free0 = smem_u32(&sh->p_free[0]);
      const uint32_t v_full0 = smem_u32(&sh->v_full[0]), v_empty0 = smem_u32(&sh->v_empty[0]);
      uint32_t pb = 0, p_par = 0, vs = 0, v_par = 0;
      for (int c = 0; c < per_walk; ++c) {
        const uint32_t t = NT == 2 ? ((uint32_t)c & 1u) : 0u;
        mbar_wait_lean(p_full0 + pb * 8u, p_par, abort_flag);
        if (t == 0) mbar_wait_lean(v_full0 + vs * 8u, v_par, abort_flag);
        tc_fence_after();
        const uint32_t a_tmem = tmem_base + SATC_TMEM_P + pb * 64u, b_lo = v_lo + vs * (uint32_t)(Cfg::TILE >> 4);
        const uint32_t d_tmem = tmem_base + Cfg::TMEM_O + t * Cfg::DP;
        const uint32_t acc0 = c >= NT ? 1u : 0u;  // the first key block starts the accumulator
#pragma unroll
        for (int kstep = 0; kstep < SATC_BK / 16; ++kstep)
          mma_f16_ts(d_tmem, a_tmem + (uint32_t)(kstep * 8), b_lo + (uint32_t)((kstep * 2048) >> 4), HI, IDESC_PV,
                     kstep > 0 ? 1u : acc0);
        if (t == NT - 1) {
          mma_commit_addr(v_empty0 + vs * 8u);
          if (++vs == (uint32_t)VST) {
            vs = 0;
            v_par ^= 1u;
          }
        }
        mma_commit_addr(p_free0 + pb * 8u);
        if (++pb == (uint32_t)PST) {
          pb = 0;
          p_par ^= 1u;
        }
        if ((c & 7) == 7 && *abort_flag) break;
      }
      mma_commit_addr(smem_u32(&sh->o_full));
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ softmax / quantizer warps
    const int q = warp & 3, cp = warp >> 2;
    const int row = q * 32 + lane;  // row of a query tile
    const uint32_t t_lane = tmem_base + ((uint32_t)(q * 32) << 16);
    const float scale = a.qk_scale_log2;
    const unsigned long long nscale2 = pack_f32x2(-scale, -scale);
    const unsigned long long one2 = pack_f32x2(1.f, 1.f);
    const unsigned long long magic2 = pack_f32x2(12582912.0f, 12582912.0f);
    const uint32_t L = (1u << a.bits) - 1u;
    const uint32_t code_top = 0x4B400000u + L;                                 // bits of 1.5 * 2^23 + last code
    const uint32_t p_top = 0x4B400000u + min(L, (uint32_t)AT_CODE_CAP);       // ... + last code with a non-zero fp16 weight
    float m_raw[NT], m2[NT], base[NT];
    unsigned long long zsum2[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      m_raw[t] = -INFINITY;
      m2[t] = 0.f;
      base[t] = 0.f;
      zsum2[t] = 0ull;
    }
    uint32_t g = 0, c = 0;  // score tiles / codes-walk tiles seen so far
    for (int w = 0; w < N_WALKS; ++w) {
      const bool walk_max = (w == 0), walk_codes = (w == N_WALKS - 1);
      for (int j = 0; j < nb; ++j) {
        const int valid = a.nk - j * SATC_BK - cp * 32;  // this warp's columns below `valid` are real keys
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          const uint32_t sb = g & 1u;
          // After a time-out every wait returns at once and the loops run to their ends on whatever the
          // buffers hold (an error is recorded): no warp leaves early, so the named barriers below are
          // always reached by all 16 warps.
          mbar_wait_lean(smem_u32(&sh->s_full[sb]), (g >> 1) & 1u, abort_flag);
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
          ++g;
          if (valid < 32) {
#pragma unroll
            for (int i = 0; i < 32; ++i)
              if (i >= valid) r[i] = 0xFF800000u;  // -inf
          }
          if (walk_max) {
            float mx0 = m_raw[t], mx1 = -INFINITY;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              mx0 = fmaxf(mx0, __uint_as_float(r[i]));
              mx1 = fmaxf(mx1, __uint_as_float(r[i + 1]));
            }
            m_raw[t] = fmaxf(mx0, mx1);
          } else if (!walk_codes) {
            // row sums with the final maximum (fixed scale: the codes need them first)
            float z0 = 0.f, z1 = 0.f;
#pragma unroll
            for (int i = 0; i < 32; i += 2) {
              z0 += ex2_approx(fmaf(__uint_as_float(r[i]), scale, -m2[t]));
              z1 += ex2_approx(fmaf(__uint_as_float(r[i + 1]), scale, -m2[t]));
            }
            zsum2[t] = pack_f32x2(__uint_as_float((uint32_t)zsum2[t]) + z0, __uint_as_float((uint32_t)(zsum2[t] >> 32)) + z1);
          } else {
            const uint32_t pb = c % PST;
            const int64_t code_row =
                (((int64_t)b * a.H + h) * a.nq + row0 + t * SATC_BQ + row) * a.nk + j * SATC_BK + cp * 32;
            const unsigned long long base2 = pack_f32x2(base[t], base[t]);
            uint32_t pk[16];
            unsigned long long zs = zsum2[t];
            {
#pragma unroll
              for (int i = 0; i < 32; i += 2) {
                // x = base - t * scale >= 0 up to rounding (the row maximum has code 0); -inf logits (keys
                // beyond nk) give +inf, which the integer minimum below clamps to the last code
                unsigned long long x2 = fma_f32x2(pack_f32x2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), nscale2, base2);
                float x0, x1;
                unpack_f32x2(x2, x0, x1);
                if (!FIXED) {
                  // 2^(t - max) = 2^-x for the row sum
                  zs = fma_f32x2(pack_f32x2(ex2_approx(-x0), ex2_approx(-x1)), one2, zs);
                } else {
                  x2 = pack_f32x2(fmaxf(x0, 0.f), fmaxf(x1, 0.f));  // a fixed scale can lie below a score
                }
                // rint by adding 1.5 * 2^23: the low bits of the sum are the integer
                float y0, y1;
                unpack_f32x2(fma_f32x2(x2, one2, magic2), y0, y1);
                const uint32_t b0 = __float_as_uint(y0), b1 = __float_as_uint(y1);
                if (CODES) {
                  r[i] = min(b0, code_top) & 0xFFu;
                  r[i + 1] = min(b1, code_top) & 0xFFu;
                }
                // 2^(14 - code) as fp32 bits: (127 + 14) << 23 minus code << 23 (the bits of 1.5 * 2^23 shift out)
                const float p0 = __uint_as_float(0x46800000u - (min(b0, p_top) << 23));
                const float p1 = __uint_as_float(0x46800000u - (min(b1, p_top) << 23));
                const __half2 ph = __floats2half2_rn(p0, p1);
                pk[i >> 1] = *reinterpret_cast<const uint32_t*>(&ph);  // key i in the low half
              }
            }
            zsum2[t] = zs;
            // the P tile's previous product must have read it
            mbar_wait_lean(smem_u32(&sh->p_free[pb]), ((c / PST) & 1u) ^ 1u, abort_flag);
            __syncwarp();
            tmem_st16(t_lane + SATC_TMEM_P + pb * 64u + cp * 16u, pk);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->p_full[pb]);
            ++c;
            if (CODES && row0 + t * SATC_BQ + row < a.nq) {
#pragma unroll
              for (int i = 0; i < 32; ++i)
                if (i < valid) a.codes_out[code_row + i] = (uint8_t)r[i];
            }
          }
        }
      }
      if (walk_max) {
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          if (t > 0) named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);  // the exchange buffer is read out
          mpart[cp * SATC_BQ + row] = m_raw[t];
          named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
          m_raw[t] = fmaxf(fmaxf(mpart[row], mpart[SATC_BQ + row]), fmaxf(mpart[2 * SATC_BQ + row], mpart[3 * SATC_BQ + row]));
          m2[t] = m_raw[t] * scale;
          base[t] = m2[t];  // row maximum as scale: log2 s + max + log2 sum = max
        }
      } else if (!walk_codes) {
        const float log2_fixed = log2f(fmaxf(__ldg(a.fixed_scale + b), 1.17549435e-38f));
#pragma unroll
        for (int t = 0; t < NT; ++t) {
          if (t > 0) named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
          zpart[cp * SATC_BQ + row] = __uint_as_float((uint32_t)zsum2[t]) + __uint_as_float((uint32_t)(zsum2[t] >> 32));
          named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
          const float z = (zpart[row] + zpart[SATC_BQ + row]) + (zpart[2 * SATC_BQ + row] + zpart[3 * SATC_BQ + row]);
          base[t] = log2_fixed + m2[t] + log2f(z);
        }
      }
    }
    float s_row[NT];
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      if (FIXED) {
        s_row[t] = fmaxf(__ldg(a.fixed_scale + b), 1.17549435e-38f);
      } else {
        if (t > 0) named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
        zpart[cp * SATC_BQ + row] = __uint_as_float((uint32_t)zsum2[t]) + __uint_as_float((uint32_t)(zsum2[t] >> 32));
        named_bar_sync(1, SATC_SOFTMAX_WARPS * 32);
        s_row[t] = 1.0f / ((zpart[row] + zpart[SATC_BQ + row]) + (zpart[2 * SATC_BQ + row] + zpart[3 * SATC_BQ + row]));
      }
      s_row[t] *= 6.103515625e-05f;  // 2^-14
    }
    mbar_wait_lean(smem_u32(&sh->o_full), 0, abort_flag);
    __syncwarp();
    tc_fence_after();
#pragma unroll
    for (int t = 0; t < NT; ++t) {
      const int orow = row0 + t * SATC_BQ + row;
      __half* o_row = a.O + (((int64_t)b * a.nq + orow) * a.H + h) * D;
      for (int ch = cp; ch < D / 8; ch += 4) {
        uint32_t o[8];
        tmem_ld8(t_lane + Cfg::TMEM_O + t * Cfg::DP + ch * 8, o);
        tmem_ld_wait();
        __half2 oh[4];
#pragma unroll
        for (int i = 0; i < 4; ++i)
          oh[i] = __floats2half2_rn(s_row[t] * __uint_as_float(o[2 * i]), s_row[t] * __uint_as_float(o[2 * i + 1]));
        if (orow < a.nq) *(reinterpret_cast<uint4*>(o_row) + ch) = *reinterpret_cast<const uint4*>(oh);
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
static dgq_status launch_self_attn2(const CUtensorMap& tmQ, const CUtensorMap& tmK, const CUtensorMap& tmV,
                                       const SelfAttnArgs& a, unsigned grid, cudaStream_t stream) {
  using Cfg = SaTcCfg<D>;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(self_attn_logq_kernel<D, FIXED, CODES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                     Cfg::SMEM));
    if (dev < 64) attr_set[dev] = true;
  }
  DGQ_CUDA_OK(launch_pdl(self_attn_logq_kernel<D, FIXED, CODES>, dim3(grid), dim3(SATC_THREADS), (size_t)Cfg::SMEM, stream,
                         tmQ, tmK, tmV, a));
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

template <int D>
static dgq_status launch_self_attn(const SelfAttnArgs& a, cudaStream_t stream) {
  SelfAttnArgs aa = a;
  aa.n_row_blocks = (a.nq + SATC_BQ * SaTcCfg<D>::NT - 1) / (SATC_BQ * SaTcCfg<D>::NT);
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
    return a.codes_out ? launch_self_attn2<D, true, true>(tmQ, tmK, tmV, aa, g, stream)
                       : launch_self_attn2<D, true, false>(tmQ, tmK, tmV, aa, g, stream);
  return a.codes_out ? launch_self_attn2<D, false, true>(tmQ, tmK, tmV, aa, g, stream)
                     : launch_self_attn2<D, false, false>(tmQ, tmK, tmV, aa, g, stream);
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
  switch (d) {
    case 40: return launch_self_attn<40>(a, st);
    case 64: return launch_self_attn<64>(a, st);
    case 80: return launch_self_attn<80>(a, st);
    case 128: return launch_self_attn<128>(a, st);
    default: return launch_self_attn<160>(a, st);
  }
}

// Cross-attention with log2-quantized softmax scores (Eq. 3, Eq. 8, Eq. 9).
//
// The scale of Eq. 8 is a maximum over a whole prompt, which every row then needs, so the work
// is two kernels on one stream:
//   phase 1  logits Q K^T (tensor cores, fp32 accumulate), per-row softmax statistics
//            (row maximum and log2 of the row sum, in base-2 logits) and the largest
//            off-<start> log2-score of the CTA's rows, one partial maximum per CTA (no atomics,
//            nothing to initialise: every partial is written before the next kernel reads it);
//   phase 2  the scale of the scope = the largest of its CTAs' partial maxima (a contiguous run
//            of at most B H ceil(nq / rows per CTA) floats, read once per CTA from L2);
//            the same logits again (bit-identical), codes in the log domain
//            code = clamp(rint(log2 s - log2 A_ij), 0, 2^b - 1) with no transcendental per score,
//            2^-code built by writing the exponent field, A_hat V on tensor cores, and the
//            <start> column added as a separate fp32 rank-1 term A_i0 V_0.
// One CTA = one (prompt, head, block of query rows); 8 warps, each owning 16 or 32 rows.  K and
// V^T of the head sit in shared memory (column 0 of V^T zeroed: the <start> key never enters the
// quantized product).  Every warp stages its Q rows in shared memory with coalesced 128-bit loads
// and writes its O rows back the same way.  HBM traffic: Q and O once (the second read of Q is
// served by L2), K and V once per CTA from L2.
#pragma once

#include <cooperative_groups.h>

#include "common.cuh"

namespace dgq {

constexpr int AT_WARPS = 8;
constexpr int AT_THREADS = AT_WARPS * 32;
constexpr float AT_P_SHIFT = 14.0f;  // A_hat / s is held in fp16 as 2^(14 - code)
constexpr float AT_CODE_CAP = 40.0f; // 2^(14 - 40) is below half the smallest fp16: codes beyond it give 0

template <int D, int NKP>
struct AttnCfg {
  static constexpr int DP = (D + 15) / 16 * 16;   // features padded to the MMA K step
  static constexpr int KS = DP / 16;
  static constexpr int LDK = DP + 8;              // row pitch of K and of a Q / O slab (halfs): conflict-free
  static constexpr int LDV = NKP * 16 + 8;        // row pitch of V^T (halfs)
  static constexpr int MT = (D <= 64 && NKP <= 5) ? 2 : 1;  // 16-row tiles per warp (register budget)
  static constexpr int WROWS = 16 * MT;
  static constexpr int ROWS = AT_WARPS * WROWS;   // query rows per CTA
  static constexpr int NT = 2 * NKP;              // 8-key tiles
  static constexpr int SM_K = NKP * 16 * LDK * 2;
  static constexpr int SM_Q = AT_WARPS * WROWS * LDK * 2;
  static constexpr int SM_V = D * LDV * 2 + D * 4;
  static constexpr int SMEM1 = SM_K + SM_Q;
  static constexpr int SMEM2 = SM_K + SM_Q + SM_V;
};

struct AttnArgs {
  const __half* Q;
  const __half* K;
  const __half* V;
  __half* O;
  int B, H, nq, nk, d, bits, gran;
  int v_bits;              // 0: V as given; else V_hat = linear quantizer (Eq. 1, Eq. 6) over the head's [nk, d] slab
  float qk_scale_log2;     // log2(e) / sqrt(d)
  float* part;             // workspace: log2 of the largest off-<start> score of every phase-1 CTA [B][H][row blocks]
  float2* stats;           // workspace: (row max, log2 row sum) [B][H][nq]
  const float* fixed_scale;
  float* scale_out;
  uint8_t* codes_out;
  int n_row_blocks;
};

__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

__device__ __forceinline__ void mma_f16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                        uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ int scope_index(const AttnArgs& a, int b, int h) {
  return a.gran == DGQ_SCALE_PER_PROMPT ? b : (a.gran == DGQ_SCALE_PER_PROMPT_HEAD ? b * a.H + h : 0);
}

// K of one head into shared memory, rows and features beyond the real ones zero.  The loads are
// issued first (into registers) and stored later, so that other loads can be put in between and
// all their latencies overlap.
template <int D, int NKP>
struct KStage {
  static constexpr int VEC = AttnCfg<D, NKP>::LDK / 8;  // 16-byte pieces per row, padding included
  static constexpr int N = (NKP * 16 * VEC + AT_THREADS - 1) / AT_THREADS;
};
template <int D, int NKP>
__device__ __forceinline__ void load_k(const AttnArgs& a, int b, int h, uint4 (&x)[KStage<D, NKP>::N]) {
  constexpr int VEC = KStage<D, NKP>::VEC;
#pragma unroll
  for (int e = 0; e < KStage<D, NKP>::N; ++e) {
    const int i = threadIdx.x + e * AT_THREADS;
    const int j = i / VEC, v = i - j * VEC;
    x[e] = make_uint4(0, 0, 0, 0);
    if (j < a.nk && v < D / 8)
      x[e] = __ldg(reinterpret_cast<const uint4*>(a.K + (((int64_t)b * a.nk + j) * a.H + h) * D) + v);
  }
}
template <int D, int NKP>
__device__ __forceinline__ void store_k(const uint4 (&x)[KStage<D, NKP>::N], __half* sK) {
  constexpr int VEC = KStage<D, NKP>::VEC;
#pragma unroll
  for (int e = 0; e < KStage<D, NKP>::N; ++e) {
    const int i = threadIdx.x + e * AT_THREADS;
    const int j = i / VEC, v = i - j * VEC;
    if (i < NKP * 16 * VEC) *reinterpret_cast<uint4*>(sK + j * AttnCfg<D, NKP>::LDK + v * 8) = x[e];
  }
}

// The warp's query rows into its slab, rows beyond the valid ones and features beyond D zero.
template <int D, int NKP>
__device__ __forceinline__ void stage_q(const __half* q_base, int64_t q_stride, int rows_valid, __half* slab) {
  using Cfg = AttnCfg<D, NKP>;
  constexpr int VEC = Cfg::DP / 8;
  constexpr int N = (Cfg::WROWS * VEC + 31) / 32;
  const int lane = threadIdx.x & 31;
  uint4 x[N];  // all loads in flight before the first store
#pragma unroll
  for (int e = 0; e < N; ++e) {
    const int i = lane + e * 32;
    const int r = i / VEC, v = i - r * VEC;
    x[e] = make_uint4(0, 0, 0, 0);
    if (i < Cfg::WROWS * VEC && r < rows_valid && v < D / 8)
      x[e] = __ldg(reinterpret_cast<const uint4*>(q_base + r * q_stride) + v);
  }
#pragma unroll
  for (int e = 0; e < N; ++e) {
    const int i = lane + e * 32;
    const int r = i / VEC, v = i - r * VEC;
    if (i < Cfg::WROWS * VEC) *reinterpret_cast<uint4*>(slab + r * Cfg::LDK + v * 8) = x[e];
  }
  __syncwarp();
}

// Four 8 x 8 fp16 matrices from shared memory: lane l gives the address of row l % 8 of matrix l / 8 (16 bytes,
// 16-byte aligned); register i of every lane holds its two elements of matrix i in the MMA fragment layout.
__device__ __forceinline__ void ldmatrix_x4(uint32_t (&x)[4], const __half* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(x[0]), "=r"(x[1]), "=r"(x[2]), "=r"(x[3])
               : "r"(smem_u32(row)));
}
__device__ __forceinline__ void ldmatrix_x2(uint32_t (&x)[2], const __half* row) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(x[0]), "=r"(x[1]) : "r"(smem_u32(row)));
}

// Base-2 logits of the warp's rows against all keys.  S[mt][nt][0..1]: row 16 mt + lane/4, keys
// 8 nt + 2 (lane%4) + {0,1}; S[mt][nt][2..3]: row + 8.  Keys >= nk get -inf.
template <int D, int NKP>
__device__ __forceinline__ void logits_warp(const AttnArgs& a, const __half* slab, const __half* sK,
                                            float (&S)[AttnCfg<D, NKP>::MT][2 * NKP][4]) {
  using Cfg = AttnCfg<D, NKP>;
  const int lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) S[mt][nt][i] = 0.f;
  // fragment addresses of this lane: matrix lane / 8, row lane % 8.  A: matrices (rows 0-7 | 8-15) x (k 0-7 | 8-15);
  // B: matrices (keys of tile nt | nt + 1) x (k 0-7 | 8-15) -- the key rows of K are the columns of the operand.
  const int lm = lane >> 3, lr = lane & 7;
  const __half* a_row = slab + ((lm & 1) * 8 + lr) * Cfg::LDK + (lm >> 1) * 8;
  const __half* b_row = sK + ((lm >> 1) * 8 + lr) * Cfg::LDK + (lm & 1) * 8;
#pragma unroll
  for (int kk = 0; kk < Cfg::KS; ++kk) {
    uint32_t af[Cfg::MT][4];
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt) ldmatrix_x4(af[mt], a_row + mt * 16 * Cfg::LDK + kk * 16);
#pragma unroll
    for (int nt = 0; nt < Cfg::NT; nt += 2) {
      uint32_t bf[4];
      ldmatrix_x4(bf, b_row + nt * 8 * Cfg::LDK + kk * 16);
#pragma unroll
      for (int mt = 0; mt < Cfg::MT; ++mt) {
        mma_f16(S[mt][nt], af[mt][0], af[mt][1], af[mt][2], af[mt][3], bf[0], bf[1]);
        mma_f16(S[mt][nt + 1], af[mt][0], af[mt][1], af[mt][2], af[mt][3], bf[2], bf[3]);
      }
    }
  }
#pragma unroll
  for (int nt = 0; nt < Cfg::NT; ++nt) {
    if (nt * 8 + 8 <= a.nk) {  // the whole 8-key tile is real (the same answer in every lane)
#pragma unroll
      for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) S[mt][nt][i] *= a.qk_scale_log2;
    } else {
#pragma unroll
      for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int key = nt * 8 + 2 * c + (i & 1);
          S[mt][nt][i] = key < a.nk ? S[mt][nt][i] * a.qk_scale_log2 : -INFINITY;
        }
    }
  }
}

template <int D, int NKP>
__global__ void __launch_bounds__(AT_THREADS, 2) attn_phase1_kernel(const AttnArgs a) {
  using Cfg = AttnCfg<D, NKP>;
  extern __shared__ __align__(16) unsigned char at_smem[];
  __half* sK = reinterpret_cast<__half*>(at_smem);
  __half* sQ = reinterpret_cast<__half*>(at_smem + Cfg::SM_K);
  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int row0 = rb * Cfg::ROWS + warp * Cfg::WROWS;
  const int rows_valid = min(Cfg::WROWS, a.nq - row0);
  const int64_t q_stride = (int64_t)a.H * D;
  __half* slab = sQ + warp * Cfg::WROWS * Cfg::LDK;
  pdl_launch_dependents();
  pdl_wait();  // Q, K, V (and, in the second pass, the first pass's statistics) may come from earlier kernels
  uint4 xk[KStage<D, NKP>::N];
  load_k<D, NKP>(a, b, h, xk);
  if (rows_valid > 0) stage_q<D, NKP>(a.Q + (((int64_t)b * a.nq + row0) * a.H + h) * D, q_stride, rows_valid, slab);
  store_k<D, NKP>(xk, sK);
  __syncthreads();
  float best = -INFINITY;
  if (rows_valid > 0) {
    float S[Cfg::MT][Cfg::NT][4];
    logits_warp<D, NKP>(a, slab, sK, S);
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {  // hi = 0: row r, hi = 1: row r + 8
        float tmax = -INFINITY, trest = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const float t = S[mt][nt][hi * 2 + i];
            if (nt == 0 && i == 0) {
              tmax = fmaxf(tmax, t);
              if (c != 0) trest = fmaxf(trest, t);  // key 0 (lane c == 0) is the <start> column
            } else {
              trest = fmaxf(trest, t);
            }
          }
        tmax = fmaxf(tmax, trest);
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        trest = fmaxf(trest, __shfl_xor_sync(0xffffffffu, trest, 1));
        trest = fmaxf(trest, __shfl_xor_sync(0xffffffffu, trest, 2));
        float z = 0.f;
#pragma unroll
        for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
          for (int i = 0; i < 2; ++i) z += ex2_approx(S[mt][nt][hi * 2 + i] - tmax);
        z += __shfl_xor_sync(0xffffffffu, z, 1);
        z += __shfl_xor_sync(0xffffffffu, z, 2);
        const float lz = log2f(z);
        const int row = mt * 16 + r + hi * 8;
        if (row < rows_valid) {
          if (c == 0) a.stats[((int64_t)b * a.H + h) * a.nq + row0 + row] = make_float2(tmax, lz);
          best = fmaxf(best, (trest - tmax) - lz);  // log2 of the row's largest off-<start> score
        }
      }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
  __shared__ float best_w[AT_WARPS];
  if (lane == 0) best_w[warp] = best;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < AT_WARPS; ++w) best = fmaxf(best, best_w[w]);
    a.part[((int64_t)b * a.H + h) * a.n_row_blocks + rb] = best;
  }
}

template <int D, int NKP, bool CODES>
__global__ void __launch_bounds__(AT_THREADS, 2) attn_phase2_kernel(const AttnArgs a) {
  using Cfg = AttnCfg<D, NKP>;
  constexpr int NT_O = D / 8;
  extern __shared__ __align__(16) unsigned char at_smem[];
  __half* sK = reinterpret_cast<__half*>(at_smem);
  __half* sQ = reinterpret_cast<__half*>(at_smem + Cfg::SM_K);
  __half* sVt = reinterpret_cast<__half*>(at_smem + Cfg::SM_K + Cfg::SM_Q);  // [D][LDV], column 0 zero
  float* sV0 = reinterpret_cast<float*>(sVt + D * Cfg::LDV);                 // [D] the <start> value row
  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int row0 = rb * Cfg::ROWS + warp * Cfg::WROWS;
  const int rows_valid = min(Cfg::WROWS, a.nq - row0);
  const int64_t q_stride = (int64_t)a.H * D;
  __half* slab = sQ + warp * Cfg::WROWS * Cfg::LDK;
  pdl_launch_dependents();
  pdl_wait();  // Q, K, V (and, in the second pass, the first pass's statistics) may come from earlier kernels
  uint4 xk[KStage<D, NKP>::N];
  load_k<D, NKP>(a, b, h, xk);
  // V^T: 128-bit loads of 8 features of one key, written transposed; keys >= nk and key 0 are zero.
  // Consecutive lanes take consecutive keys of the same 8 features, so that the transposed 2-byte stores
  // of a warp fall into consecutive words of one V^T row (the head's V slab is a few KB and sits in L2,
  // so the strided reads cost little).  K, V and Q are all requested before anything is written, so
  // their latencies overlap.
  constexpr int NV = (NKP * 16 * (D / 8) + AT_THREADS - 1) / AT_THREADS;
  uint4 xv[NV];
#pragma unroll
  for (int e = 0; e < NV; ++e) {
    const int i = threadIdx.x + e * AT_THREADS;
    const int v = i / (NKP * 16), j = i - v * (NKP * 16);
    xv[e] = make_uint4(0, 0, 0, 0);
    if (j < a.nk && v < D / 8)
      xv[e] = __ldg(reinterpret_cast<const uint4*>(a.V + (((int64_t)b * a.nk + j) * a.H + h) * D) + v);
  }
  // The scope's scale: its CTAs' partial maxima lie next to each other (row blocks of a head, heads of a
  // prompt, prompts of the call); each thread takes a strided share, the warps meet after the barrier below.
  __shared__ float part_w[AT_WARPS];
  if (!a.fixed_scale) {
    const int per_head = a.n_row_blocks;
    const int64_t first = a.gran == DGQ_SCALE_PER_PROMPT ? (int64_t)b * a.H * per_head
                          : (a.gran == DGQ_SCALE_PER_PROMPT_HEAD ? ((int64_t)b * a.H + h) * per_head : 0);
    const int count = a.gran == DGQ_SCALE_PER_PROMPT ? a.H * per_head
                      : (a.gran == DGQ_SCALE_PER_PROMPT_HEAD ? per_head : a.B * a.H * per_head);
    float m = -INFINITY;
    for (int i = threadIdx.x; i < count; i += AT_THREADS) m = fmaxf(m, __ldg(a.part + first + i));
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) part_w[warp] = m;
  }
  if (rows_valid > 0) stage_q<D, NKP>(a.Q + (((int64_t)b * a.nq + row0) * a.H + h) * D, q_stride, rows_valid, slab);
  store_k<D, NKP>(xk, sK);
  // Quantized value operand: range of the head's slab (every CTA of the head derives the same
  // parameters), codes decided in fp32, de-quantized as s (q - Z); rows j >= 1 become the fp16
  // operand of the product, row 0 stays fp32.
  float v_s = 0.f, v_inv = 0.f, v_Zf = 0.f, v_L = 0.f;
  if (a.v_bits) {
    __shared__ float v_red[2 * (AT_THREADS / 32)];
    float lo = INFINITY, hi = -INFINITY;
#pragma unroll
    for (int ev = 0; ev < NV; ++ev) {
      const int i = threadIdx.x + ev * AT_THREADS;
      if (i % (NKP * 16) < a.nk && i < NKP * 16 * (D / 8)) {
        const __half* xh = reinterpret_cast<const __half*>(&xv[ev]);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float f = __half2float(xh[e]);
          lo = fminf(lo, f);
          hi = fmaxf(hi, f);
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) {
      v_red[warp] = lo;
      v_red[AT_THREADS / 32 + warp] = hi;
    }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < AT_THREADS / 32; ++w) {
      lo = fminf(lo, v_red[w]);
      hi = fmaxf(hi, v_red[AT_THREADS / 32 + w]);
    }
    int v_Z;
    group_params(lo, hi, a.v_bits, v_s, v_inv, v_Z);
    v_Zf = (float)v_Z;
    v_L = (float)((1 << a.v_bits) - 1);
  }
#pragma unroll
  for (int ev = 0; ev < NV; ++ev) {
    const int i = threadIdx.x + ev * AT_THREADS;
    if (i >= NKP * 16 * (D / 8)) continue;
    const int v = i / (NKP * 16), j = i - v * (NKP * 16);
    const __half* xh = reinterpret_cast<const __half*>(&xv[ev]);
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      f[e] = __half2float(xh[e]);
      if (a.v_bits && j < a.nk)
        f[e] = __fmul_rn(v_s, __fsub_rn((float)quantize_code(f[e], v_inv, v_Zf, v_L), v_Zf));
    }
    if (j == 0) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        sV0[v * 8 + e] = f[e];
        sVt[(v * 8 + e) * Cfg::LDV] = __float2half(0.f);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) sVt[(v * 8 + e) * Cfg::LDV + j] = __float2half_rn(f[e]);
    }
  }
  __syncthreads();
  const int scope = scope_index(a, b, h);
  float log2s;
  if (a.fixed_scale) {
    log2s = log2f(fmaxf(__ldg(a.fixed_scale + scope), 1.17549435e-38f));
  } else {
    log2s = part_w[0];
#pragma unroll
    for (int w = 1; w < AT_WARPS; ++w) log2s = fmaxf(log2s, part_w[w]);
  }
  if (a.scale_out && threadIdx.x == 0 && rb == 0 &&
      (a.gran == DGQ_SCALE_PER_PROMPT_HEAD || (a.gran == DGQ_SCALE_PER_PROMPT && h == 0) || (b == 0 && h == 0)))
    a.scale_out[scope] = exp2f(log2s);
  if (rows_valid <= 0) return;
  float S[Cfg::MT][Cfg::NT][4];
  logits_warp<D, NKP>(a, slab, sK, S);
  __syncwarp();  // the slab is reused for the output rows below

  const float Lf = (float)((1 << a.bits) - 1);
  const float Lcap = fminf(Lf, AT_CODE_CAP);
  uint32_t pa[Cfg::MT][NKP][4];  // A fragments of A_hat / s * 2^14 for the second product
  float a0[Cfg::MT][2];          // the <start> score of rows r and r + 8
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      const int row = min(mt * 16 + r + hi * 8, rows_valid - 1);
      const float2 st = __ldg(a.stats + ((int64_t)b * a.H + h) * a.nq + row0 + row);
      const float base = log2s + st.x + st.y;  // code = rint(base - t)
      float start = ex2_approx(S[mt][0][hi * 2] - st.x - st.y);  // meaningful on the lane with c == 0
      a0[mt][hi] = __shfl_sync(0xffffffffu, start, lane & ~3);
#pragma unroll
      for (int nt = 0; nt < Cfg::NT; ++nt) {
        float p[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float t = S[mt][nt][hi * 2 + i];
          // rint by adding 1.5 * 2^23: the low bits of the sum are the integer.  -inf logits (padding
          // keys) clamp to the cap; their V^T columns are zero, as is the <start> column.
          const float x = fminf(fmaxf(base - t, 0.f), CODES ? Lf : Lcap);
          const uint32_t bits = __float_as_uint(x + 12582912.0f);  // 0x4B400000 + code
          if (CODES) {
            const int key = nt * 8 + 2 * c + i;
            const int orow = mt * 16 + r + hi * 8;
            if (key >= 1 && key < a.nk && orow < rows_valid)
              a.codes_out[(((int64_t)b * a.H + h) * a.nq + row0 + orow) * (a.nk - 1) + key - 1] = (uint8_t)(bits & 0xFFu);
          }
          // 2^(14 - code) as an fp32 exponent field: (127 + 14 - code) << 23, where the shift drops the
          // 0x4B400000 of `bits` (its low 9 bits are zero).  Without the code output x is already held
          // to the cap, beyond which the product would convert to an fp16 zero anyway.
          const uint32_t capped = CODES ? min(bits, 0x4B400000u + (uint32_t)AT_CODE_CAP) : bits;
          p[i] = __uint_as_float(((127u + (uint32_t)AT_P_SHIFT) << 23) - (capped << 23));
        }
        const __half2 ph = __floats2half2_rn(p[0], p[1]);
        pa[mt][nt >> 1][(nt & 1) * 2 + hi] = *reinterpret_cast<const uint32_t*>(&ph);
      }
    }
  float acc[Cfg::MT][NT_O][4];
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
  {
    const int lm = lane >> 3, lr = lane & 7;  // matrix and row this lane addresses
    const __half* v_row = sVt + ((lm >> 1) * 8 + lr) * Cfg::LDV + (lm & 1) * 8;
#pragma unroll
    for (int kk = 0; kk < NKP; ++kk) {
#pragma unroll
      for (int nt = 0; nt + 1 < NT_O; nt += 2) {
        uint32_t bf[4];
        ldmatrix_x4(bf, v_row + nt * 8 * Cfg::LDV + kk * 16);
#pragma unroll
        for (int mt = 0; mt < Cfg::MT; ++mt) {
          mma_f16(acc[mt][nt], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], bf[0], bf[1]);
          mma_f16(acc[mt][nt + 1], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], bf[2], bf[3]);
        }
      }
      if (NT_O & 1) {  // the last 8 features alone (lanes 16-31 repeat the addresses of lanes 0-15, unused)
        uint32_t bf[2];
        ldmatrix_x2(bf, v_row - (lm >> 1) * 8 * Cfg::LDV + (NT_O - 1) * 8 * Cfg::LDV + kk * 16);
#pragma unroll
        for (int mt = 0; mt < Cfg::MT; ++mt)
          mma_f16(acc[mt][NT_O - 1], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], bf[0], bf[1]);
      }
    }
  }
  // O = A_i0 V_0 + s 2^-14 acc, staged in the warp's slab and written with 128-bit stores
  const float s_out = exp2f(log2s - AT_P_SHIFT);
#pragma unroll
  for (int nt = 0; nt < NT_O; ++nt) {
    const int col = nt * 8 + 2 * c;
    const float2 v0 = *reinterpret_cast<const float2*>(sV0 + col);
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const float ox = fmaf(a0[mt][hi], v0.x, s_out * acc[mt][nt][hi * 2]);
        const float oy = fmaf(a0[mt][hi], v0.y, s_out * acc[mt][nt][hi * 2 + 1]);
        *reinterpret_cast<__half2*>(slab + (mt * 16 + r + hi * 8) * Cfg::LDK + col) = __floats2half2_rn(ox, oy);
      }
  }
  __syncwarp();
  __half* o_base = a.O + (((int64_t)b * a.nq + row0) * a.H + h) * D;
  for (int i = lane; i < Cfg::WROWS * (D / 8); i += 32) {
    const int rr = i / (D / 8), v = i - rr * (D / 8);
    if (rr < rows_valid)
      *(reinterpret_cast<uint4*>(o_base + rr * q_stride) + v) = *reinterpret_cast<const uint4*>(slab + rr * Cfg::LDK + v * 8);
  }
}

// The two passes as one kernel: the logits and the row statistics stay in registers while the CTAs exchange
// their maxima through the workspace and meet at the grid barrier, so Q K^T, the K / Q staging and the
// statistics round trip happen once.  Launched cooperatively (every CTA resident) when the scale is dynamic;
// with a fixed scale no CTA waits for another and the launch is an ordinary one.
template <int D, int NKP, bool CODES>
__global__ void __launch_bounds__(AT_THREADS, 2) attn_fused_kernel(const AttnArgs a) {
  using Cfg = AttnCfg<D, NKP>;
  constexpr int NT_O = D / 8;
  extern __shared__ __align__(16) unsigned char at_smem[];
  __half* sK = reinterpret_cast<__half*>(at_smem);
  __half* sQ = reinterpret_cast<__half*>(at_smem + Cfg::SM_K);
  __half* sVt = reinterpret_cast<__half*>(at_smem + Cfg::SM_K + Cfg::SM_Q);  // [D][LDV], column 0 zero
  float* sV0 = reinterpret_cast<float*>(sVt + D * Cfg::LDV);                 // [D] the <start> value row
  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int row0 = rb * Cfg::ROWS + warp * Cfg::WROWS;
  const int rows_valid = min(Cfg::WROWS, a.nq - row0);
  const int64_t q_stride = (int64_t)a.H * D;
  __half* slab = sQ + warp * Cfg::WROWS * Cfg::LDK;
  pdl_launch_dependents();
  pdl_wait();  // Q, K, V may come from earlier kernels
  uint4 xk[KStage<D, NKP>::N];
  load_k<D, NKP>(a, b, h, xk);
  // V^T: 128-bit loads of 8 features of one key, written transposed; keys >= nk and key 0 are zero.
  // Consecutive lanes take consecutive keys of the same 8 features, so that the transposed 2-byte stores
  // of a warp fall into consecutive words of one V^T row (the head's V slab is a few KB and sits in L2,
  // so the strided reads cost little).  K, V and Q are all requested before anything is written, so
  // their latencies overlap.
  // V is first needed after the scope's CTAs have met.  A slab of a few registers is requested up front with K
  // and Q; a larger one is requested once the logits are there (the registers of the Q K^T fragments are free
  // again) and arrives while the row statistics and the meeting take their time.
  constexpr int NV = (NKP * 16 * (D / 8) + AT_THREADS - 1) / AT_THREADS;
  constexpr bool V_EARLY = NV <= 2;
  uint4 xv[NV];
  auto request_v = [&]() {
#pragma unroll
    for (int e = 0; e < NV; ++e) {
      const int i = threadIdx.x + e * AT_THREADS;
      const int v = i / (NKP * 16), j = i - v * (NKP * 16);
      xv[e] = make_uint4(0, 0, 0, 0);
      if (j < a.nk && v < D / 8)
        xv[e] = __ldg(reinterpret_cast<const uint4*>(a.V + (((int64_t)b * a.nk + j) * a.H + h) * D) + v);
    }
  };
  if (V_EARLY) request_v();
  // The scope's scale: its CTAs' partial maxima lie next to each other (row blocks of a head, heads of a
  // prompt, prompts of the call); each thread takes a strided share, the warps meet after the barrier below.
  __shared__ float part_w[AT_WARPS];
  if (rows_valid > 0) stage_q<D, NKP>(a.Q + (((int64_t)b * a.nq + row0) * a.H + h) * D, q_stride, rows_valid, slab);
  store_k<D, NKP>(xk, sK);
  __syncthreads();
  const int scope = scope_index(a, b, h);
  // Logits once; they stay in registers across the meeting of the scope's CTAs.
  float S[Cfg::MT][Cfg::NT][4];
  float st_max[Cfg::MT][2], st_lz[Cfg::MT][2];  // row maximum and log2 of the row sum, rows r and r + 8 of every tile
  float best = -INFINITY;
  if (rows_valid > 0) logits_warp<D, NKP>(a, slab, sK, S);
  if (!V_EARLY) request_v();
  if (rows_valid > 0) {
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        float tmax = -INFINITY, trest = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
          for (int i = 0; i < 2; ++i) {
            const float t = S[mt][nt][hi * 2 + i];
            if (nt == 0 && i == 0) {
              tmax = fmaxf(tmax, t);
              if (c != 0) trest = fmaxf(trest, t);  // key 0 (lane c == 0) is the <start> column
            } else {
              trest = fmaxf(trest, t);
            }
          }
        tmax = fmaxf(tmax, trest);
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
        tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
        trest = fmaxf(trest, __shfl_xor_sync(0xffffffffu, trest, 1));
        trest = fmaxf(trest, __shfl_xor_sync(0xffffffffu, trest, 2));
        float z = 0.f;
#pragma unroll
        for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
          for (int i = 0; i < 2; ++i) z += ex2_approx(S[mt][nt][hi * 2 + i] - tmax);
        z += __shfl_xor_sync(0xffffffffu, z, 1);
        z += __shfl_xor_sync(0xffffffffu, z, 2);
        const float lz = log2f(z);
        st_max[mt][hi] = tmax;
        st_lz[mt][hi] = lz;
        if (mt * 16 + r + hi * 8 < rows_valid) best = fmaxf(best, (trest - tmax) - lz);  // log2 of the row's largest off-<start> score
      }
  }
  __syncwarp();  // the slab is reused for the output rows below
  // The scope's scale: every CTA leaves its maximum in its own word, all CTAs of the grid meet (the grid is
  // launched cooperatively, so all of them are resident and the runtime's grid barrier applies), then every CTA
  // reduces the words of its scope.  The V^T operand is staged between the store and the meeting.
  if (!a.fixed_scale) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
    if (lane == 0) part_w[warp] = best;
    __syncthreads();
    if (threadIdx.x == 0) {
#pragma unroll
      for (int w = 1; w < AT_WARPS; ++w) best = fmaxf(best, part_w[w]);
      a.part[((int64_t)b * a.H + h) * a.n_row_blocks + rb] = best;
    }
  }
  // Quantized value operand: range of the head's slab (every CTA of the head derives the same
  // parameters), codes decided in fp32, de-quantized as s (q - Z); rows j >= 1 become the fp16
  // operand of the product, row 0 stays fp32.
  float v_s = 0.f, v_inv = 0.f, v_Zf = 0.f, v_L = 0.f;
  if (a.v_bits) {
    __shared__ float v_red[2 * (AT_THREADS / 32)];
    float lo = INFINITY, hi = -INFINITY;
#pragma unroll
    for (int ev = 0; ev < NV; ++ev) {
      const int i = threadIdx.x + ev * AT_THREADS;
      if (i % (NKP * 16) < a.nk && i < NKP * 16 * (D / 8)) {
        const __half* xh = reinterpret_cast<const __half*>(&xv[ev]);
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float f = __half2float(xh[e]);
          lo = fminf(lo, f);
          hi = fmaxf(hi, f);
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, o));
      hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, o));
    }
    if (lane == 0) {
      v_red[warp] = lo;
      v_red[AT_THREADS / 32 + warp] = hi;
    }
    __syncthreads();
#pragma unroll
    for (int w = 0; w < AT_THREADS / 32; ++w) {
      lo = fminf(lo, v_red[w]);
      hi = fmaxf(hi, v_red[AT_THREADS / 32 + w]);
    }
    int v_Z;
    group_params(lo, hi, a.v_bits, v_s, v_inv, v_Z);
    v_Zf = (float)v_Z;
    v_L = (float)((1 << a.v_bits) - 1);
  }
#pragma unroll
  for (int ev = 0; ev < NV; ++ev) {
    const int i = threadIdx.x + ev * AT_THREADS;
    if (i >= NKP * 16 * (D / 8)) continue;
    const int v = i / (NKP * 16), j = i - v * (NKP * 16);
    const __half* xh = reinterpret_cast<const __half*>(&xv[ev]);
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      f[e] = __half2float(xh[e]);
      if (a.v_bits && j < a.nk)
        f[e] = __fmul_rn(v_s, __fsub_rn((float)quantize_code(f[e], v_inv, v_Zf, v_L), v_Zf));
    }
    if (j == 0) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        sV0[v * 8 + e] = f[e];
        sVt[(v * 8 + e) * Cfg::LDV] = __float2half(0.f);
      }
    } else {
#pragma unroll
      for (int e = 0; e < 8; ++e) sVt[(v * 8 + e) * Cfg::LDV + j] = __float2half_rn(f[e]);
    }
  }
  float log2s;
  if (a.fixed_scale) {
    log2s = log2f(fmaxf(__ldg(a.fixed_scale + scope), 1.17549435e-38f));
    __syncthreads();  // V^T is staged
  } else {
    cooperative_groups::this_grid().sync();  // every CTA's maximum is written and visible; V^T is staged
    const int per_head = a.n_row_blocks;
    const int64_t first = a.gran == DGQ_SCALE_PER_PROMPT ? (int64_t)b * a.H * per_head
                          : (a.gran == DGQ_SCALE_PER_PROMPT_HEAD ? ((int64_t)b * a.H + h) * per_head : 0);
    const int count = a.gran == DGQ_SCALE_PER_PROMPT ? a.H * per_head
                      : (a.gran == DGQ_SCALE_PER_PROMPT_HEAD ? per_head : a.B * a.H * per_head);
    float m = -INFINITY;
    for (int i = threadIdx.x; i < count; i += AT_THREADS) m = fmaxf(m, __ldcg(a.part + first + i));  // written by this grid: L2
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    if (lane == 0) part_w[warp] = m;  // (free again: the grid barrier is also a barrier of the CTA)
    __syncthreads();
    log2s = part_w[0];
#pragma unroll
    for (int w = 1; w < AT_WARPS; ++w) log2s = fmaxf(log2s, part_w[w]);
  }
  if (a.scale_out && threadIdx.x == 0 && rb == 0 &&
      (a.gran == DGQ_SCALE_PER_PROMPT_HEAD || (a.gran == DGQ_SCALE_PER_PROMPT && h == 0) || (b == 0 && h == 0)))
    a.scale_out[scope] = exp2f(log2s);
  if (rows_valid <= 0) return;

  const float Lf = (float)((1 << a.bits) - 1);
  const float Lcap = fminf(Lf, AT_CODE_CAP);
  uint32_t pa[Cfg::MT][NKP][4];  // A fragments of A_hat / s * 2^14 for the second product
  float a0[Cfg::MT][2];          // the <start> score of rows r and r + 8
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      const float2 st = make_float2(st_max[mt][hi], st_lz[mt][hi]);
      const float base = log2s + st.x + st.y;  // code = rint(base - t)
      float start = ex2_approx(S[mt][0][hi * 2] - st.x - st.y);  // meaningful on the lane with c == 0
      a0[mt][hi] = __shfl_sync(0xffffffffu, start, lane & ~3);
#pragma unroll
      for (int nt = 0; nt < Cfg::NT; ++nt) {
        float p[2];
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float t = S[mt][nt][hi * 2 + i];
          // rint by adding 1.5 * 2^23: the low bits of the sum are the integer.  -inf logits (padding
          // keys) clamp to the cap; their V^T columns are zero, as is the <start> column.
          const float x = fminf(fmaxf(base - t, 0.f), CODES ? Lf : Lcap);
          const uint32_t bits = __float_as_uint(x + 12582912.0f);  // 0x4B400000 + code
          if (CODES) {
            const int key = nt * 8 + 2 * c + i;
            const int orow = mt * 16 + r + hi * 8;
            if (key >= 1 && key < a.nk && orow < rows_valid)
              a.codes_out[(((int64_t)b * a.H + h) * a.nq + row0 + orow) * (a.nk - 1) + key - 1] = (uint8_t)(bits & 0xFFu);
          }
          // 2^(14 - code) as an fp32 exponent field: (127 + 14 - code) << 23, where the shift drops the
          // 0x4B400000 of `bits` (its low 9 bits are zero).  Without the code output x is already held
          // to the cap, beyond which the product would convert to an fp16 zero anyway.
          const uint32_t capped = CODES ? min(bits, 0x4B400000u + (uint32_t)AT_CODE_CAP) : bits;
          p[i] = __uint_as_float(((127u + (uint32_t)AT_P_SHIFT) << 23) - (capped << 23));
        }
        const __half2 ph = __floats2half2_rn(p[0], p[1]);
        pa[mt][nt >> 1][(nt & 1) * 2 + hi] = *reinterpret_cast<const uint32_t*>(&ph);
      }
    }
  float acc[Cfg::MT][NT_O][4];
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
  {
    const int lm = lane >> 3, lr = lane & 7;  // matrix and row this lane addresses
    const __half* v_row = sVt + ((lm >> 1) * 8 + lr) * Cfg::LDV + (lm & 1) * 8;
#pragma unroll
    for (int kk = 0; kk < NKP; ++kk) {
#pragma unroll
      for (int nt = 0; nt + 1 < NT_O; nt += 2) {
        uint32_t bf[4];
        ldmatrix_x4(bf, v_row + nt * 8 * Cfg::LDV + kk * 16);
#pragma unroll
        for (int mt = 0; mt < Cfg::MT; ++mt) {
          mma_f16(acc[mt][nt], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], bf[0], bf[1]);
          mma_f16(acc[mt][nt + 1], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], bf[2], bf[3]);
        }
      }
      if (NT_O & 1) {  // the last 8 features alone (lanes 16-31 repeat the addresses of lanes 0-15, unused)
        uint32_t bf[2];
        ldmatrix_x2(bf, v_row - (lm >> 1) * 8 * Cfg::LDV + (NT_O - 1) * 8 * Cfg::LDV + kk * 16);
#pragma unroll
        for (int mt = 0; mt < Cfg::MT; ++mt)
          mma_f16(acc[mt][NT_O - 1], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], bf[0], bf[1]);
      }
    }
  }
  // O = A_i0 V_0 + s 2^-14 acc, staged in the warp's slab and written with 128-bit stores
  const float s_out = exp2f(log2s - AT_P_SHIFT);
#pragma unroll
  for (int nt = 0; nt < NT_O; ++nt) {
    const int col = nt * 8 + 2 * c;
    const float2 v0 = *reinterpret_cast<const float2*>(sV0 + col);
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const float ox = fmaf(a0[mt][hi], v0.x, s_out * acc[mt][nt][hi * 2]);
        const float oy = fmaf(a0[mt][hi], v0.y, s_out * acc[mt][nt][hi * 2 + 1]);
        *reinterpret_cast<__half2*>(slab + (mt * 16 + r + hi * 8) * Cfg::LDK + col) = __floats2half2_rn(ox, oy);
      }
  }
  __syncwarp();
  __half* o_base = a.O + (((int64_t)b * a.nq + row0) * a.H + h) * D;
  for (int i = lane; i < Cfg::WROWS * (D / 8); i += 32) {
    const int rr = i / (D / 8), v = i - rr * (D / 8);
    if (rr < rows_valid)
      *(reinterpret_cast<uint4*>(o_base + rr * q_stride) + v) = *reinterpret_cast<const uint4*>(slab + rr * Cfg::LDK + v * 8);
  }
}

// Launch with the cooperative attribute: every CTA of the grid is resident at the same time (the launch
// fails instead of running a grid that is not), which the fused kernel's meeting of CTAs relies on.
template <typename... KArgs, typename... Args>
static cudaError_t launch_cooperative(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                                      Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

template <int D, int NKP>
static dgq_status launch_attn(const AttnArgs& a, bool allow_fused, cudaStream_t stream) {
  using Cfg = AttnCfg<D, NKP>;
  constexpr int SM1 = Cfg::SMEM1;
  constexpr int SM2 = Cfg::SMEM2;
  static std::atomic<int> capacity[64];  // CTAs of the fused kernel that fit the device at once; 0 = not asked yet
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev < 0 || dev >= 64) return DGQ_ERR_UNSUPPORTED;
  if (capacity[dev].load() == 0) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_phase1_kernel<D, NKP>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM1));
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_phase2_kernel<D, NKP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM2));
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_phase2_kernel<D, NKP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM2));
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_fused_kernel<D, NKP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM2));
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_fused_kernel<D, NKP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM2));
    int n_sm = 0, per_sm0 = 0, per_sm1 = 0;
    DGQ_CUDA_OK(cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev));
    DGQ_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm0, attn_fused_kernel<D, NKP, false>, AT_THREADS, SM2));
    DGQ_CUDA_OK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm1, attn_fused_kernel<D, NKP, true>, AT_THREADS, SM2));
    capacity[dev].store(std::max(1, n_sm * std::min(per_sm0, per_sm1)));
  }
  AttnArgs aa = a;
  aa.n_row_blocks = (a.nq + Cfg::ROWS - 1) / Cfg::ROWS;
  const int grid = a.B * a.H * aa.n_row_blocks;
  if (allow_fused && (a.fixed_scale != nullptr || grid <= capacity[dev].load())) {
    // one kernel: with a fixed scale its CTAs never wait for one another; with a dynamic one they meet at the
    // grid barrier, and the launch guarantees that all of them are resident
    if (a.fixed_scale) {
      if (a.codes_out)
        DGQ_CUDA_OK(launch_pdl(attn_fused_kernel<D, NKP, true>, dim3(grid), dim3(AT_THREADS), (size_t)SM2, stream, aa));
      else
        DGQ_CUDA_OK(launch_pdl(attn_fused_kernel<D, NKP, false>, dim3(grid), dim3(AT_THREADS), (size_t)SM2, stream, aa));
    } else {
      if (a.codes_out)
        DGQ_CUDA_OK(launch_cooperative(attn_fused_kernel<D, NKP, true>, dim3(grid), dim3(AT_THREADS), (size_t)SM2, stream, aa));
      else
        DGQ_CUDA_OK(launch_cooperative(attn_fused_kernel<D, NKP, false>, dim3(grid), dim3(AT_THREADS), (size_t)SM2, stream, aa));
    }
    g_launches += 1;
    DGQ_CUDA_OK(cudaGetLastError());
    return DGQ_OK;
  }
  DGQ_CUDA_OK(launch_pdl(attn_phase1_kernel<D, NKP>, dim3(grid), dim3(AT_THREADS), (size_t)SM1, stream, aa));
  if (a.codes_out)
    DGQ_CUDA_OK(launch_pdl(attn_phase2_kernel<D, NKP, true>, dim3(grid), dim3(AT_THREADS), (size_t)SM2, stream, aa));
  else
    DGQ_CUDA_OK(launch_pdl(attn_phase2_kernel<D, NKP, false>, dim3(grid), dim3(AT_THREADS), (size_t)SM2, stream, aa));
  g_launches += 2;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

template <int D>
static dgq_status launch_attn_d(const AttnArgs& a, bool allow_fused, cudaStream_t stream) {
  if (a.nk <= 80) return launch_attn<D, 5>(a, allow_fused, stream);
  return launch_attn<D, 8>(a, allow_fused, stream);
}

// One partial maximum per CTA; the bound holds for every kernel configuration (128 or 256 rows per CTA).
static size_t attn_part_bytes(int B, int H, int nq) {
  return ((size_t)B * H * ((nq + 127) / 128) * sizeof(float) + 255) / 256 * 256;
}

}  // namespace dgq

extern "C" dgq_status dgq_cross_attn_workspace_bytes(int B, int H, int nq, int nk, int d, size_t* bytes) {
  if (!bytes || B <= 0 || H <= 0 || nq <= 0 || nk < 2 || d <= 0) return DGQ_ERR_INVALID_ARG;
  *bytes = dgq::attn_part_bytes(B, H, nq) + (size_t)B * H * nq * sizeof(float2);
  return DGQ_OK;
}

namespace dgq {
// The argument checks every cross-attention entry point makes first, in this order.
static dgq_status attn_check_args(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk, int d,
                                  int score_bits, int scale_gran, int v_bits, const void* O) {
  if (!Q || !K || !V || !O || B <= 0 || H <= 0 || nq <= 0 || d <= 0) return DGQ_ERR_INVALID_ARG;
  if (v_bits != 0 && (v_bits < 2 || v_bits > 8)) return DGQ_ERR_INVALID_ARG;
  if (nk < 2) return DGQ_ERR_INVALID_ARG;
  if (score_bits < 2 || score_bits > 8) return DGQ_ERR_INVALID_ARG;
  if (scale_gran < DGQ_SCALE_PER_PROMPT || scale_gran > DGQ_SCALE_PER_CALL) return DGQ_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return DGQ_ERR_ALIGNMENT;
  if (nk > 128 || (d != 40 && d != 64 && d != 80 && d != 128 && d != 160)) return DGQ_ERR_UNSUPPORTED;
  return DGQ_OK;
}

static dgq_status attn_run(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk, int d,
                           int score_bits, int scale_gran, const float* fixed_scale, int v_bits, void* O,
                           float* scale_out, uint8_t* codes_out, void* workspace, size_t workspace_bytes,
                           bool allow_fused, void* stream) {
  dgq_status chk = attn_check_args(Q, K, V, B, H, nq, nk, d, score_bits, scale_gran, v_bits, O);
  if (chk != DGQ_OK) return chk;
  size_t need = 0;
  dgq_cross_attn_workspace_bytes(B, H, nq, nk, d, &need);
  if (!workspace || workspace_bytes < need) return DGQ_ERR_WORKSPACE;
  if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return DGQ_ERR_ALIGNMENT;
  AttnArgs a;
  a.Q = (const __half*)Q;
  a.K = (const __half*)K;
  a.V = (const __half*)V;
  a.O = (__half*)O;
  a.B = B;
  a.H = H;
  a.nq = nq;
  a.nk = nk;
  a.d = d;
  a.bits = score_bits;
  a.gran = scale_gran;
  a.v_bits = v_bits;
  a.qk_scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)d));
  a.part = (float*)workspace;
  a.stats = (float2*)((char*)workspace + attn_part_bytes(B, H, nq));
  a.fixed_scale = fixed_scale;
  a.scale_out = scale_out;
  a.codes_out = codes_out;
  a.n_row_blocks = 0;  // set per kernel configuration at launch
  cudaStream_t st = (cudaStream_t)stream;
  switch (d) {
    case 40: return launch_attn_d<40>(a, allow_fused, st);
    case 64: return launch_attn_d<64>(a, allow_fused, st);
    case 80: return launch_attn_d<80>(a, allow_fused, st);
    case 128: return launch_attn_d<128>(a, allow_fused, st);
    default: return launch_attn_d<160>(a, allow_fused, st);
  }
}
}  // namespace dgq

extern "C" dgq_status dgq_cross_attn_logq(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk,
                                          int d, int score_bits, int scale_gran, const float* fixed_scale, void* O,
                                          float* scale_out, uint8_t* codes_out, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  return dgq::attn_run(Q, K, V, B, H, nq, nk, d, score_bits, scale_gran, fixed_scale, 0, O, scale_out, codes_out,
                       workspace, workspace_bytes, true, stream);
}

extern "C" dgq_status dgq_cross_attn_logq_qv(const void* Q, const void* K, const void* V, int B, int H, int nq,
                                             int nk, int d, int score_bits, int scale_gran, const float* fixed_scale,
                                             int v_bits, void* O, float* scale_out, uint8_t* codes_out,
                                             void* workspace, size_t workspace_bytes, void* stream) {
  if (v_bits < 2 || v_bits > 8) return DGQ_ERR_INVALID_ARG;
  return dgq::attn_run(Q, K, V, B, H, nq, nk, d, score_bits, scale_gran, fixed_scale, v_bits, O, scale_out,
                       codes_out, workspace, workspace_bytes, true, stream);
}

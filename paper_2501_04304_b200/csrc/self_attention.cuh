// Attention with log2-quantized softmax scores and no <start> column (self-attention; Sec. 3.3
// applies the log quantizer of Eq. 2 "to both self and cross-attentions"):
//     A = softmax(Q K^T / sqrt(d)),  code = clamp(rint(-log2(A / s)), 0, 2^b - 1),  O = s sum_j 2^-code_j V_j
// with s the largest score of the query row, or one fixed scale per prompt.
//
// The key axis is as long as the query axis (up to 4096), so the keys are walked in blocks of 64
// twice by the same CTA: the first walk keeps a running maximum and sum of every row (the softmax
// statistics), the second recomputes the logits, forms the codes in the log domain and multiplies
// with the block of V.  No workspace and no second kernel: with a per-row or fixed scale nothing has
// to be reduced across CTAs.  One CTA = one (prompt, head, block of query rows); K and V^T blocks
// are loaded into registers one block ahead and parked in shared memory between two CTA barriers.
// The building blocks (shared-memory layouts, warp-level MMA fragments, the fp16 exponent-field
// construction of 2^-code) are those of the cross-attention kernels.
#pragma once

#include "attention.cuh"

namespace dgq {

constexpr int SA_NKP = 4;            // 16-key pairs per block
constexpr int SA_KB = SA_NKP * 16;   // keys per block

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

// 64 keys of K starting at key0 (rows and features beyond the real ones zero) into registers / smem.
template <int D>
__device__ __forceinline__ void sa_load_k(const SelfAttnArgs& a, int b, int h, int key0,
                                          uint4 (&x)[KStage<D, SA_NKP>::N]) {
  constexpr int VEC = KStage<D, SA_NKP>::VEC;
#pragma unroll
  for (int e = 0; e < KStage<D, SA_NKP>::N; ++e) {
    const int i = threadIdx.x + e * AT_THREADS;
    const int j = i / VEC, v = i - j * VEC;
    x[e] = make_uint4(0, 0, 0, 0);
    if (i < SA_KB * VEC && key0 + j < a.nk && v < D / 8)
      x[e] = __ldg(reinterpret_cast<const uint4*>(a.K + (((int64_t)b * a.nk + key0 + j) * a.H + h) * D) + v);
  }
}

template <int D>
struct SaVStage {
  static constexpr int N = (SA_KB * (D / 8) + AT_THREADS - 1) / AT_THREADS;
};
template <int D>
__device__ __forceinline__ void sa_load_v(const SelfAttnArgs& a, int b, int h, int key0, uint4 (&x)[SaVStage<D>::N]) {
#pragma unroll
  for (int e = 0; e < SaVStage<D>::N; ++e) {
    const int i = threadIdx.x + e * AT_THREADS;
    const int j = i / (D / 8), v = i - j * (D / 8);
    x[e] = make_uint4(0, 0, 0, 0);
    if (i < SA_KB * (D / 8) && key0 + j < a.nk)
      x[e] = __ldg(reinterpret_cast<const uint4*>(a.V + (((int64_t)b * a.nk + key0 + j) * a.H + h) * D) + v);
  }
}
// V block written transposed: sVt[feature][key in block]; keys beyond nk hold zeros.
template <int D>
__device__ __forceinline__ void sa_store_vt(const uint4 (&x)[SaVStage<D>::N], __half* sVt) {
  constexpr int LDV = AttnCfg<D, SA_NKP>::LDV;
#pragma unroll
  for (int e = 0; e < SaVStage<D>::N; ++e) {
    const int i = threadIdx.x + e * AT_THREADS;
    if (i >= SA_KB * (D / 8)) continue;
    const int j = i / (D / 8), v = i - j * (D / 8);
    const __half* xh = reinterpret_cast<const __half*>(&x[e]);
#pragma unroll
    for (int q = 0; q < 8; ++q) sVt[(v * 8 + q) * LDV + j] = xh[q];
  }
}

// Base-2 logits of the warp's rows against the 64 keys in shared memory; keys >= keys_left get -inf.
template <int D>
__device__ __forceinline__ void sa_logits(const __half* slab, const __half* sK, int keys_left, float qk_scale_log2,
                                          float (&S)[AttnCfg<D, SA_NKP>::MT][2 * SA_NKP][4]) {
  using Cfg = AttnCfg<D, SA_NKP>;
  const int lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) S[mt][nt][i] = 0.f;
#pragma unroll
  for (int kk = 0; kk < Cfg::KS; ++kk) {
    uint32_t af[Cfg::MT][4];
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int i = 0; i < 4; ++i)
        af[mt][i] = *reinterpret_cast<const uint32_t*>(slab + (mt * 16 + r + (i & 1) * 8) * Cfg::LDK + kk * 16 +
                                                       2 * c + (i >> 1) * 8);
#pragma unroll
    for (int nt = 0; nt < Cfg::NT; ++nt) {
      const __half* kp = sK + (nt * 8 + r) * Cfg::LDK + kk * 16 + 2 * c;
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kp);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kp + 8);
#pragma unroll
      for (int mt = 0; mt < Cfg::MT; ++mt) mma_f16(S[mt][nt], af[mt][0], af[mt][1], af[mt][2], af[mt][3], b0, b1);
    }
  }
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int key = nt * 8 + 2 * c + (i & 1);
        S[mt][nt][i] = key < keys_left ? S[mt][nt][i] * qk_scale_log2 : -INFINITY;
      }
}

template <int D, bool CODES>
__global__ void __launch_bounds__(AT_THREADS, 1) self_attn_logq_kernel(const SelfAttnArgs a) {
  using Cfg = AttnCfg<D, SA_NKP>;
  constexpr int NT_O = D / 8;
  extern __shared__ __align__(16) unsigned char at_smem[];
  __half* sK = reinterpret_cast<__half*>(at_smem);
  __half* sQ = reinterpret_cast<__half*>(at_smem + Cfg::SM_K);
  __half* sVt = reinterpret_cast<__half*>(at_smem + Cfg::SM_K + Cfg::SM_Q);  // [D][LDV]
  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int row0 = rb * Cfg::ROWS + warp * Cfg::WROWS;
  const int rows_valid = min(Cfg::WROWS, a.nq - row0);  // may be <= 0: the warp still helps with the loads
  const int64_t q_stride = (int64_t)a.H * D;
  __half* slab = sQ + warp * Cfg::WROWS * Cfg::LDK;
  const int n_blocks = (a.nk + SA_KB - 1) / SA_KB;
  pdl_launch_dependents();
  pdl_wait();  // Q, K and V may come from earlier kernels
  uint4 xk[KStage<D, SA_NKP>::N];
  sa_load_k<D>(a, b, h, 0, xk);
  if (rows_valid > 0) stage_q<D, SA_NKP>(a.Q + (((int64_t)b * a.nq + row0) * a.H + h) * D, q_stride, rows_valid, slab);

  // ---- first walk over the keys: running maximum and sum of 2^(t - max) of every row
  float m[Cfg::MT][2], z[Cfg::MT][2];
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      m[mt][hi] = -INFINITY;
      z[mt][hi] = 0.f;
    }
  for (int kb = 0; kb < n_blocks; ++kb) {
    __syncthreads();  // everyone is done with the previous block
    store_k<D, SA_NKP>(xk, sK);
    __syncthreads();
    if (kb + 1 < n_blocks) sa_load_k<D>(a, b, h, (kb + 1) * SA_KB, xk);  // travels during the arithmetic
    if (rows_valid > 0) {
      float S[Cfg::MT][Cfg::NT][4];
      sa_logits<D>(slab, sK, a.nk - kb * SA_KB, a.qk_scale_log2, S);
#pragma unroll
      for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
          float tmax = -INFINITY;
#pragma unroll
          for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
            for (int i = 0; i < 2; ++i) tmax = fmaxf(tmax, S[mt][nt][hi * 2 + i]);
          tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
          tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
          const float mn = fmaxf(m[mt][hi], tmax);  // finite: every block holds at least one real key
          float zz = 0.f;
#pragma unroll
          for (int nt = 0; nt < Cfg::NT; ++nt)
#pragma unroll
            for (int i = 0; i < 2; ++i) zz += ex2_approx(S[mt][nt][hi * 2 + i] - mn);
          zz += __shfl_xor_sync(0xffffffffu, zz, 1);
          zz += __shfl_xor_sync(0xffffffffu, zz, 2);
          z[mt][hi] = z[mt][hi] * ex2_approx(m[mt][hi] - mn) + zz;
          m[mt][hi] = mn;
        }
    }
  }
  // code = rint(base - t) with base = log2 s + max + log2 sum; with the row maximum as scale
  // (s = 1 / sum) this is the row maximum of the logits itself
  float base[Cfg::MT][2], s_out[Cfg::MT][2];
  {
    const float log2_fixed = a.fixed_scale ? log2f(fmaxf(__ldg(a.fixed_scale + b), 1.17549435e-38f)) : 0.f;
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi) {
        const float lz = log2f(z[mt][hi]);
        const float log2s = a.fixed_scale ? log2_fixed : -lz;
        base[mt][hi] = a.fixed_scale ? log2_fixed + m[mt][hi] + lz : m[mt][hi];
        s_out[mt][hi] = exp2f(log2s - AT_P_SHIFT);
      }
  }

  // ---- second walk: codes and the product with V
  const float Lf = (float)((1 << a.bits) - 1);
  const float Lcap = fminf(Lf, AT_CODE_CAP);
  float acc[Cfg::MT][NT_O][4];
#pragma unroll
  for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt)
#pragma unroll
      for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;
  uint4 xv[SaVStage<D>::N];
  sa_load_k<D>(a, b, h, 0, xk);
  sa_load_v<D>(a, b, h, 0, xv);
  for (int kb = 0; kb < n_blocks; ++kb) {
    __syncthreads();
    store_k<D, SA_NKP>(xk, sK);
    sa_store_vt<D>(xv, sVt);
    __syncthreads();
    if (kb + 1 < n_blocks) {
      sa_load_k<D>(a, b, h, (kb + 1) * SA_KB, xk);
      sa_load_v<D>(a, b, h, (kb + 1) * SA_KB, xv);
    }
    if (rows_valid > 0) {
      float S[Cfg::MT][Cfg::NT][4];
      sa_logits<D>(slab, sK, a.nk - kb * SA_KB, a.qk_scale_log2, S);
      uint32_t pa[Cfg::MT][SA_NKP][4];  // A fragments of A_hat / s * 2^14
#pragma unroll
      for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
        for (int hi = 0; hi < 2; ++hi) {
#pragma unroll
          for (int nt = 0; nt < Cfg::NT; ++nt) {
            float p[2];
#pragma unroll
            for (int i = 0; i < 2; ++i) {
              const float t = S[mt][nt][hi * 2 + i];
              // rint by adding 1.5 * 2^23: the low bits of the sum are the integer.  -inf logits
              // (keys beyond nk) clamp to the cap; their V^T columns are zero.
              const float x = fminf(fmaxf(base[mt][hi] - t, 0.f), CODES ? Lf : Lcap);
              const int code = __float_as_int(x + 12582912.0f) - 0x4B400000;
              if (CODES) {
                const int key = kb * SA_KB + nt * 8 + 2 * c + i;
                const int orow = mt * 16 + r + hi * 8;
                if (key < a.nk && orow < rows_valid)
                  a.codes_out[(((int64_t)b * a.H + h) * a.nq + row0 + orow) * a.nk + key] = (uint8_t)code;
              }
              p[i] = __int_as_float((127 + (int)AT_P_SHIFT - min(code, (int)AT_CODE_CAP)) << 23);
            }
            const __half2 ph = __floats2half2_rn(p[0], p[1]);
            pa[mt][nt >> 1][(nt & 1) * 2 + hi] = *reinterpret_cast<const uint32_t*>(&ph);
          }
        }
#pragma unroll
      for (int kk = 0; kk < SA_NKP; ++kk)
#pragma unroll
        for (int nt = 0; nt < NT_O; ++nt) {
          const __half* vp = sVt + (nt * 8 + r) * Cfg::LDV + kk * 16 + 2 * c;
          const uint32_t b0 = *reinterpret_cast<const uint32_t*>(vp);
          const uint32_t b1 = *reinterpret_cast<const uint32_t*>(vp + 8);
#pragma unroll
          for (int mt = 0; mt < Cfg::MT; ++mt)
            mma_f16(acc[mt][nt], pa[mt][kk][0], pa[mt][kk][1], pa[mt][kk][2], pa[mt][kk][3], b0, b1);
        }
    }
  }
  if (rows_valid <= 0) return;
  // O = s 2^-14 acc, staged in the warp's slab (its Q rows are no longer needed) and written with 128-bit stores
  __syncwarp();
#pragma unroll
  for (int nt = 0; nt < NT_O; ++nt) {
    const int col = nt * 8 + 2 * c;
#pragma unroll
    for (int mt = 0; mt < Cfg::MT; ++mt)
#pragma unroll
      for (int hi = 0; hi < 2; ++hi)
        *reinterpret_cast<__half2*>(slab + (mt * 16 + r + hi * 8) * Cfg::LDK + col) =
            __floats2half2_rn(s_out[mt][hi] * acc[mt][nt][hi * 2], s_out[mt][hi] * acc[mt][nt][hi * 2 + 1]);
  }
  __syncwarp();
  __half* o_base = a.O + (((int64_t)b * a.nq + row0) * a.H + h) * D;
  for (int i = lane; i < Cfg::WROWS * (D / 8); i += 32) {
    const int rr = i / (D / 8), v = i - rr * (D / 8);
    if (rr < rows_valid)
      *(reinterpret_cast<uint4*>(o_base + rr * q_stride) + v) = *reinterpret_cast<const uint4*>(slab + rr * Cfg::LDK + v * 8);
  }
}

template <int D>
static dgq_status launch_self_attn(const SelfAttnArgs& a, cudaStream_t stream) {
  using Cfg = AttnCfg<D, SA_NKP>;
  constexpr int SM = Cfg::SMEM2;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(self_attn_logq_kernel<D, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM));
    DGQ_CUDA_OK(cudaFuncSetAttribute(self_attn_logq_kernel<D, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM));
    if (dev < 64) attr_set[dev] = true;
  }
  SelfAttnArgs aa = a;
  aa.n_row_blocks = (a.nq + Cfg::ROWS - 1) / Cfg::ROWS;
  const int64_t grid = (int64_t)a.B * a.H * aa.n_row_blocks;
  if (grid > INT_MAX) return DGQ_ERR_UNSUPPORTED;
  if (a.codes_out)
    DGQ_CUDA_OK(launch_pdl(self_attn_logq_kernel<D, true>, dim3((unsigned)grid), dim3(AT_THREADS), (size_t)SM, stream, aa));
  else
    DGQ_CUDA_OK(launch_pdl(self_attn_logq_kernel<D, false>, dim3((unsigned)grid), dim3(AT_THREADS), (size_t)SM, stream, aa));
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

}  // namespace dgq


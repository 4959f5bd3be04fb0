// Cross-attention with log2-quantized softmax scores (Eq. 3, Eq. 8, Eq. 9).
//
// The scale of Eq. 8 is a maximum over a whole prompt, which every row then needs, so the work
// is two kernels on one stream:
//   phase 1  logits Q K^T (tensor cores, fp32 accumulate), per-row softmax statistics
//            (row maximum and log2 of the row sum, in base-2 logits) and the largest
//            off-<start> log2-score of the scope, reduced with an ordered-integer atomicMax;
//   phase 2  the same logits again (bit-identical), codes in the log domain
//            code = clamp(rint(log2 s - log2 A_ij), 0, 2^b - 1) with no transcendental per score,
//            2^-code built by writing the fp16 exponent field, A_hat V on tensor cores, and the
//            <start> column added as a separate fp32 rank-1 term A_i0 V_0.
// One CTA = one (prompt, head, 128 query rows); 8 warps of 16 rows.  K and V^T of the head sit in
// shared memory.  HBM traffic: Q and O once (the second read of Q is served by L2), K and V once.
#pragma once

#include "common.cuh"

namespace dgq {

constexpr int AT_ROWS = 128;
constexpr int AT_THREADS = 256;
constexpr float AT_P_SHIFT = 14.0f;  // A_hat / s is held in fp16 as 2^(14 - code)

struct AttnArgs {
  const __half* Q;
  const __half* K;
  const __half* V;
  __half* O;
  int B, H, nq, nk, d, bits, gran;
  float qk_scale_log2;     // log2(e) / sqrt(d)
  int* smax;               // workspace: ordered-int log2 of the scale per scope
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

// Base-2 logits of 16 query rows against all keys: S[nt][0..1] = row lane/4, keys 8 nt + 2 (lane%4) + {0,1};
// S[nt][2..3] = row lane/4 + 8.  Keys >= nk get -inf.
template <int D, int NKP>
__device__ __forceinline__ void logits_16rows(const AttnArgs& a, const __half* q_base, int64_t q_stride,
                                              int rows_valid, const __half* sK, float (&S)[2 * NKP][4]) {
  constexpr int DP = (D + 15) / 16 * 16;
  constexpr int KS = DP / 16;
  constexpr int LDK = DP + 8;  // padded row length of K in shared memory (halfs): conflict-free fragment reads
  const int lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
#pragma unroll
  for (int nt = 0; nt < 2 * NKP; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) S[nt][i] = 0.f;
#pragma unroll
  for (int kk = 0; kk < KS; ++kk) {
    uint32_t af[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int row = r + (i & 1) * 8;
      const int col = kk * 16 + 2 * c + (i >> 1) * 8;
      af[i] = (row < rows_valid && col < D)
                  ? __ldg(reinterpret_cast<const uint32_t*>(q_base + row * q_stride + col))
                  : 0u;
    }
#pragma unroll
    for (int nt = 0; nt < 2 * NKP; ++nt) {
      const __half* kp = sK + (nt * 8 + r) * LDK + kk * 16 + 2 * c;
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(kp);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(kp + 8);
      mma_f16(S[nt], af[0], af[1], af[2], af[3], b0, b1);
    }
  }
#pragma unroll
  for (int nt = 0; nt < 2 * NKP; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int key = nt * 8 + 2 * c + (i & 1);
      S[nt][i] = key < a.nk ? S[nt][i] * a.qk_scale_log2 : -INFINITY;
    }
}

template <int D, int NKP>
__device__ __forceinline__ void stage_k(const AttnArgs& a, int b, int h, __half* sK) {
  constexpr int DP = (D + 15) / 16 * 16;
  constexpr int LDK = DP + 8;
  // zero everything (padding keys and features), then copy the head's keys with 128-bit loads
  for (int i = threadIdx.x; i < NKP * 16 * LDK / 8; i += AT_THREADS) reinterpret_cast<uint4*>(sK)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  const int vec = D / 8;
  for (int i = threadIdx.x; i < a.nk * vec; i += AT_THREADS) {
    const int j = i / vec, v = i - j * vec;
    const uint4 x = __ldg(reinterpret_cast<const uint4*>(a.K + (((int64_t)b * a.nk + j) * a.H + h) * D) + v);
    *reinterpret_cast<uint4*>(sK + j * LDK + v * 8) = x;
  }
}

template <int D, int NKP>
__global__ void __launch_bounds__(AT_THREADS) attn_phase1_kernel(const AttnArgs a) {
  constexpr int DP = (D + 15) / 16 * 16;
  constexpr int LDK = DP + 8;
  extern __shared__ __align__(16) unsigned char at_smem[];
  __half* sK = reinterpret_cast<__half*>(at_smem);  // [NKP * 16][LDK]
  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  stage_k<D, NKP>(a, b, h, sK);
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int row0 = rb * AT_ROWS + warp * 16;
  const int rows_valid = min(16, a.nq - row0);
  float best = -INFINITY;
  if (rows_valid > 0) {
    const int64_t q_stride = (int64_t)a.H * D;
    const __half* q_base = a.Q + (((int64_t)b * a.nq + row0) * a.H + h) * D;
    float S[2 * NKP][4];
    logits_16rows<D, NKP>(a, q_base, q_stride, rows_valid, sK, S);
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {  // hi = 0: row r, hi = 1: row r + 8
      float tmax = -INFINITY, trest = -INFINITY;
#pragma unroll
      for (int nt = 0; nt < 2 * NKP; ++nt)
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          const float t = S[nt][hi * 2 + i];
          tmax = fmaxf(tmax, t);
          const bool is_start = (nt == 0) && (c == 0) && (i == 0);
          if (!is_start) trest = fmaxf(trest, t);
        }
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 1));
      tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, 2));
      trest = fmaxf(trest, __shfl_xor_sync(0xffffffffu, trest, 1));
      trest = fmaxf(trest, __shfl_xor_sync(0xffffffffu, trest, 2));
      float z = 0.f;
#pragma unroll
      for (int nt = 0; nt < 2 * NKP; ++nt)
#pragma unroll
        for (int i = 0; i < 2; ++i) z += ex2_approx(S[nt][hi * 2 + i] - tmax);
      z += __shfl_xor_sync(0xffffffffu, z, 1);
      z += __shfl_xor_sync(0xffffffffu, z, 2);
      const float lz = log2f(z);
      const int row = r + hi * 8;
      if (row < rows_valid) {
        if (c == 0) a.stats[((int64_t)b * a.H + h) * a.nq + row0 + row] = make_float2(tmax, lz);
        best = fmaxf(best, (trest - tmax) - lz);  // log2 of the row's largest off-<start> score
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) best = fmaxf(best, __shfl_xor_sync(0xffffffffu, best, o));
  if (lane == 0 && best > -INFINITY && a.fixed_scale == nullptr)
    atomicMax(&a.smax[scope_index(a, b, h)], float_to_ordered(best));
}

template <int D, int NKP>
__global__ void __launch_bounds__(AT_THREADS) attn_phase2_kernel(const AttnArgs a) {
  constexpr int DP = (D + 15) / 16 * 16;
  constexpr int LDK = DP + 8;
  constexpr int LDV = NKP * 16 + 8;  // padded row length of V^T in shared memory (halfs)
  constexpr int NT_O = D / 8;
  extern __shared__ __align__(16) unsigned char at_smem[];
  __half* sK = reinterpret_cast<__half*>(at_smem);  // [NKP * 16][LDK]
  __half* sVt = sK + NKP * 16 * LDK;                // [D][LDV]
  const int blk = blockIdx.x;
  const int rb = blk % a.n_row_blocks;
  const int h = (blk / a.n_row_blocks) % a.H;
  const int b = blk / (a.n_row_blocks * a.H);
  stage_k<D, NKP>(a, b, h, sK);
  for (int i = threadIdx.x; i < D * LDV / 8; i += AT_THREADS) reinterpret_cast<uint4*>(sVt)[i] = make_uint4(0, 0, 0, 0);
  __syncthreads();
  for (int i = threadIdx.x; i < a.nk * D; i += AT_THREADS) {
    const int j = i / D, f = i - j * D;
    sVt[f * LDV + j] = a.V[(((int64_t)b * a.nk + j) * a.H + h) * D + f];
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int r = lane >> 2, c = lane & 3;
  const int row0 = rb * AT_ROWS + warp * 16;
  const int rows_valid = min(16, a.nq - row0);
  const int scope = scope_index(a, b, h);
  float log2s;
  if (a.fixed_scale)
    log2s = log2f(fmaxf(__ldg(a.fixed_scale + scope), 1.17549435e-38f));
  else
    log2s = ordered_to_float(a.smax[scope]);
  if (a.scale_out && threadIdx.x == 0 && rb == 0 &&
      (a.gran == DGQ_SCALE_PER_PROMPT_HEAD || (a.gran == DGQ_SCALE_PER_PROMPT && h == 0) || (b == 0 && h == 0)))
    a.scale_out[scope] = exp2f(log2s);
  if (rows_valid <= 0) return;
  const int64_t q_stride = (int64_t)a.H * D;
  const __half* q_base = a.Q + (((int64_t)b * a.nq + row0) * a.H + h) * D;
  float S[2 * NKP][4];
  logits_16rows<D, NKP>(a, q_base, q_stride, rows_valid, sK, S);

  const float Lf = (float)((1 << a.bits) - 1);
  uint32_t pa[NKP][4];  // A fragments of A_hat / s * 2^14 for the second product
  float a0[2];          // the <start> score of rows r and r + 8
#pragma unroll
  for (int hi = 0; hi < 2; ++hi) {
    const int row = min(r + hi * 8, rows_valid - 1);
    const float2 st = a.stats[((int64_t)b * a.H + h) * a.nq + row0 + row];
    const float base = log2s + st.x + st.y;  // code = rint(base - t)
    float start = ex2_approx(S[0][hi * 2] - st.x - st.y);  // meaningful on the lane with c == 0
    start = __shfl_sync(0xffffffffu, start, lane & ~3);
    a0[hi] = start;
#pragma unroll
    for (int nt = 0; nt < 2 * NKP; ++nt) {
      uint32_t packed = 0;
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const float t = S[nt][hi * 2 + i];
        const int key = nt * 8 + 2 * c + i;
        // -inf logits (padding keys) give +inf -> the last code; they are dropped below
        const float code_f = fminf(fmaxf(rintf(base - t), 0.f), Lf);
        const int code = (int)code_f;
        uint32_t bits16 = 0;
        if (key >= 1 && key < a.nk) {
          const int e = (int)AT_P_SHIFT - code;  // exponent of 2^(14 - code)
          bits16 = e >= -14 ? (uint32_t)(e + 15) << 10 : (e >= -24 ? 1u << (e + 24) : 0u);
          if (a.codes_out && (r + hi * 8) < rows_valid)
            a.codes_out[(((int64_t)b * a.H + h) * a.nq + row0 + r + hi * 8) * (a.nk - 1) + key - 1] = (uint8_t)code;
        }
        packed |= bits16 << (16 * i);
      }
      pa[nt >> 1][(nt & 1) * 2 + hi] = packed;
    }
  }
  float acc[NT_O][4];
#pragma unroll
  for (int nt = 0; nt < NT_O; ++nt)
#pragma unroll
    for (int i = 0; i < 4; ++i) acc[nt][i] = 0.f;
#pragma unroll
  for (int kk = 0; kk < NKP; ++kk)
#pragma unroll
    for (int nt = 0; nt < NT_O; ++nt) {
      const __half* vp = sVt + (nt * 8 + r) * LDV + kk * 16 + 2 * c;
      const uint32_t b0 = *reinterpret_cast<const uint32_t*>(vp);
      const uint32_t b1 = *reinterpret_cast<const uint32_t*>(vp + 8);
      mma_f16(acc[nt], pa[kk][0], pa[kk][1], pa[kk][2], pa[kk][3], b0, b1);
    }
  const float s_out = exp2f(log2s - AT_P_SHIFT);
  __half* o_base = a.O + (((int64_t)b * a.nq + row0) * a.H + h) * D;
#pragma unroll
  for (int nt = 0; nt < NT_O; ++nt) {
    const int col = nt * 8 + 2 * c;
    const float v0x = __half2float(sVt[col * LDV]), v0y = __half2float(sVt[(col + 1) * LDV]);
#pragma unroll
    for (int hi = 0; hi < 2; ++hi) {
      const int row = r + hi * 8;
      if (row < rows_valid) {
        const float ox = fmaf(a0[hi], v0x, s_out * acc[nt][hi * 2]);
        const float oy = fmaf(a0[hi], v0y, s_out * acc[nt][hi * 2 + 1]);
        *reinterpret_cast<__half2*>(o_base + row * q_stride + col) = __floats2half2_rn(ox, oy);
      }
    }
  }
}

template <int D, int NKP>
static dgq_status launch_attn(const AttnArgs& a, cudaStream_t stream) {
  constexpr int DP = (D + 15) / 16 * 16;
  constexpr int SM1 = NKP * 16 * (DP + 8) * 2;
  constexpr int SM2 = SM1 + D * (NKP * 16 + 8) * 2;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_phase1_kernel<D, NKP>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM1));
    DGQ_CUDA_OK(cudaFuncSetAttribute(attn_phase2_kernel<D, NKP>, cudaFuncAttributeMaxDynamicSharedMemorySize, SM2));
    if (dev < 64) attr_set[dev] = true;
  }
  const int grid = a.B * a.H * a.n_row_blocks;
  attn_phase1_kernel<D, NKP><<<grid, AT_THREADS, SM1, stream>>>(a);
  attn_phase2_kernel<D, NKP><<<grid, AT_THREADS, SM2, stream>>>(a);
  g_launches += 2;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}

template <int D>
static dgq_status launch_attn_d(const AttnArgs& a, cudaStream_t stream) {
  if (a.nk <= 80) return launch_attn<D, 5>(a, stream);
  return launch_attn<D, 8>(a, stream);
}

static size_t attn_smax_bytes(int B, int H) { return ((size_t)B * H * sizeof(int) + 255) / 256 * 256; }

}  // namespace dgq

extern "C" dgq_status dgq_cross_attn_workspace_bytes(int B, int H, int nq, int nk, int d, size_t* bytes) {
  if (!bytes || B <= 0 || H <= 0 || nq <= 0 || nk < 2 || d <= 0) return DGQ_ERR_INVALID_ARG;
  *bytes = dgq::attn_smax_bytes(B, H) + (size_t)B * H * nq * sizeof(float2);
  return DGQ_OK;
}

extern "C" dgq_status dgq_cross_attn_logq(const void* Q, const void* K, const void* V, int B, int H, int nq, int nk,
                                          int d, int score_bits, int scale_gran, const float* fixed_scale, void* O,
                                          float* scale_out, uint8_t* codes_out, void* workspace,
                                          size_t workspace_bytes, void* stream) {
  using namespace dgq;
  if (!Q || !K || !V || !O || B <= 0 || H <= 0 || nq <= 0 || d <= 0) return DGQ_ERR_INVALID_ARG;
  if (nk < 2) return DGQ_ERR_INVALID_ARG;
  if (score_bits < 2 || score_bits > 8) return DGQ_ERR_INVALID_ARG;
  if (scale_gran < DGQ_SCALE_PER_PROMPT || scale_gran > DGQ_SCALE_PER_CALL) return DGQ_ERR_INVALID_ARG;
  if (!aligned16(Q) || !aligned16(K) || !aligned16(V) || !aligned16(O)) return DGQ_ERR_ALIGNMENT;
  if (nk > 128 || (d != 40 && d != 64 && d != 80 && d != 128 && d != 160)) return DGQ_ERR_UNSUPPORTED;
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
  a.qk_scale_log2 = (float)(1.4426950408889634 / std::sqrt((double)d));
  a.smax = (int*)workspace;
  a.stats = (float2*)((char*)workspace + attn_smax_bytes(B, H));
  a.fixed_scale = fixed_scale;
  a.scale_out = scale_out;
  a.codes_out = codes_out;
  a.n_row_blocks = (nq + AT_ROWS - 1) / AT_ROWS;
  cudaStream_t st = (cudaStream_t)stream;
  // 0x80 bytes decode to about -3.4e38 in the ordered-integer encoding: "no score seen yet"
  DGQ_CUDA_OK(cudaMemsetAsync(a.smax, 0x80, attn_smax_bytes(B, H), st));
  switch (d) {
    case 40: return launch_attn_d<40>(a, st);
    case 64: return launch_attn_d<64>(a, st);
    case 80: return launch_attn_d<80>(a, st);
    case 128: return launch_attn_d<128>(a, st);
    default: return launch_attn_d<160>(a, st);
  }
}

// Activation quantizer: Eq. 1 with the per-cell parameters of Eq. 6, fused with the channel
// permutation into the padded, group-contiguous code layout the GEMM reads.
//
// One warp owns one or two rows at a time and never synchronises with the rest of the CTA: it
// stages its rows in shared memory with coalesced 128-bit loads, then every lane takes 16-code
// chunks of the output (all 16 codes of a chunk belong to one channel group, since groups are
// padded to multiples of 32 positions), gathers their source channels through the permutation
// table and writes one 16-byte vector, so a warp writes 512 contiguous bytes.
// Dynamic-token mode first reduces the range of every (row, group) cell: a lane reduces its
// chunks, lanes that share a cell merge through shared-memory atomics on order-preserving
// integer keys, and one lane per cell derives (s, 1/s, Z).
// HBM traffic: 2 B read + 1 B written per element (+ 8 B per (token, group) in dynamic mode).
#pragma once

#include "groups.cuh"

namespace dgq {

constexpr int QA_THREADS = 256;
constexpr int QA_WARPS = QA_THREADS / 32;

struct QuantArgs {
  const __half* X;
  uint8_t* Xq;
  int64_t M, ld;
  int C, K_pad, G, P, bits, rows_per_warp;
  int dynamic, centred;
  const int16_t* perm;
  const uint8_t* chunk_group;
  const int32_t* row_group;
  const float* inv_scale;  // static: table row of the timestep [R][G]
  const int32_t* zp;
  float* dyn_scale;        // dynamic: outputs [M][G]
  int32_t* dyn_zp;
};

// The 16 source channels of one chunk (two 128-bit loads of int16 indices; -1 = padding).
__device__ __forceinline__ void load_chunk_perm(const int16_t* perm, int ch, int (&c)[16]) {
  const uint4 lo = *reinterpret_cast<const uint4*>(perm + ch * 16);
  const uint4 hi = *(reinterpret_cast<const uint4*>(perm + ch * 16) + 1);
  const uint32_t w[8] = {lo.x, lo.y, lo.z, lo.w, hi.x, hi.y, hi.z, hi.w};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    c[2 * j] = (int)(int16_t)(w[j] & 0xFFFFu);
    c[2 * j + 1] = (int)(int16_t)(w[j] >> 16);
  }
}

__global__ void __launch_bounds__(QA_THREADS, 4) quantize_act_kernel(const QuantArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int n_chunks = a.K_pad >> 4;
  // layout: perm [K_pad] int16 | chunk_group [n_chunks] u8 | per warp: rows [rpw][C] fp16, cells [rpw][G] x 4 ints
  int16_t* perm_s = reinterpret_cast<int16_t*>(smem_raw);
  uint8_t* cg_s = reinterpret_cast<uint8_t*>(perm_s + a.K_pad);
  const int head = (a.K_pad * 2 + n_chunks + 15) & ~15;
  const int rpw = a.rows_per_warp;
  const int warp_bytes = ((rpw * a.C * 2 + 15) & ~15) + rpw * a.G * 16;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  unsigned char* wbase = smem_raw + head + warp * warp_bytes;
  __half* rows_s = reinterpret_cast<__half*>(wbase);
  int* cell_lo = reinterpret_cast<int*>(wbase + ((rpw * a.C * 2 + 15) & ~15));
  int* cell_hi = cell_lo + rpw * a.G;
  float* cell_inv = reinterpret_cast<float*>(cell_hi + rpw * a.G);
  int* cell_z = reinterpret_cast<int*>(cell_inv + rpw * a.G);

  for (int i = threadIdx.x; i < a.K_pad / 8; i += QA_THREADS)
    reinterpret_cast<uint4*>(perm_s)[i] = __ldg(reinterpret_cast<const uint4*>(a.perm) + i);
  for (int i = threadIdx.x; i < n_chunks; i += QA_THREADS) cg_s[i] = a.chunk_group[i];
  __syncthreads();

  const int vec_per_row = a.C >> 3;
  const float Lf = (float)((1 << a.bits) - 1);
  const int64_t warps_total = (int64_t)gridDim.x * QA_WARPS;
  for (int64_t row0 = ((int64_t)blockIdx.x * QA_WARPS + warp) * rpw; row0 < a.M; row0 += warps_total * rpw) {
    const int rows = (int)min((int64_t)rpw, a.M - row0);
    // Row loads in batches of four 128-bit pieces per lane: every load of a batch is issued before
    // the first store, so the memory latency is paid once per batch and not once per piece.
    {
      const int n_vec = rows * vec_per_row;
      for (int v0 = 0; v0 < n_vec; v0 += 4 * 32) {
        uint4 x[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = v0 + e * 32 + lane;
          if (i < n_vec) {
            const int r = i / vec_per_row, v = i - r * vec_per_row;
            x[e] = __ldg(reinterpret_cast<const uint4*>(a.X + (row0 + r) * a.ld) + v);
          }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const int i = v0 + e * 32 + lane;
          if (i < n_vec) reinterpret_cast<uint4*>(rows_s)[i] = x[e];  // rows are packed: pitch C halfs
        }
      }
    }
    if (a.dynamic)
      for (int i = lane; i < rows * a.G; i += 32) {
        cell_lo[i] = INT_MAX;
        cell_hi[i] = INT_MIN;
      }
    __syncwarp();

    if (a.dynamic) {
      for (int r = 0; r < rows; ++r) {
        const __half* row = rows_s + r * a.C;
        for (int ch = lane; ch < n_chunks; ch += 32) {
          float lo = INFINITY, hi = -INFINITY;
          int cidx[16];
          load_chunk_perm(perm_s, ch, cidx);
#pragma unroll
          for (int j = 0; j < 16; ++j)
            if (cidx[j] >= 0) {
              const float v = __half2float(row[cidx[j]]);
              lo = fminf(lo, v);
              hi = fmaxf(hi, v);
            }
          if (lo <= hi) {
            const int g = cg_s[ch];
            atomicMin(&cell_lo[r * a.G + g], float_to_ordered(lo));
            atomicMax(&cell_hi[r * a.G + g], float_to_ordered(hi));
          }
        }
      }
      __syncwarp();
      for (int i = lane; i < rows * a.G; i += 32) {
        float lo = 0.f, hi = 0.f;
        if (cell_lo[i] != INT_MAX) {
          lo = ordered_to_float(cell_lo[i]);
          hi = ordered_to_float(cell_hi[i]);
        }
        float s, inv_s;
        int Z;
        group_params(lo, hi, a.bits, s, inv_s, Z);
        cell_inv[i] = inv_s;
        cell_z[i] = Z;
        const int r = i / a.G, g = i - r * a.G;
        a.dyn_scale[(row0 + r) * a.G + g] = s;
        a.dyn_zp[(row0 + r) * a.G + g] = Z;
      }
      __syncwarp();
    }

    for (int r = 0; r < rows; ++r) {
      const __half* row = rows_s + r * a.C;
      const int rg = a.dynamic ? 0 : a.row_group[(row0 + r) % a.P];
      uint8_t* out = a.Xq + (row0 + r) * a.K_pad;
      for (int ch = lane; ch < n_chunks; ch += 32) {
        const int g = cg_s[ch];
        float inv_s;
        int Z;
        if (a.dynamic) {
          inv_s = cell_inv[r * a.G + g];
          Z = cell_z[r * a.G + g];
        } else {
          inv_s = __ldg(a.inv_scale + rg * a.G + g);
          Z = __ldg(a.zp + rg * a.G + g);
        }
        const float Zf = (float)Z;
        const int pad_code = a.centred ? 0 : min(max(Z, 0), (1 << a.bits) - 1);
        const int sub = a.centred ? Z : 0;
        uint32_t w[4];
        int cidx[16];
        load_chunk_perm(perm_s, ch, cidx);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t word = 0;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int c = cidx[q * 4 + j];
            int code = pad_code;
            if (c >= 0) code = quantize_code(__half2float(row[c]), inv_s, Zf, Lf) - sub;
            word |= (uint32_t)(code & 0xFF) << (8 * j);
          }
          w[q] = word;
        }
        *reinterpret_cast<uint4*>(out + ch * 16) = make_uint4(w[0], w[1], w[2], w[3]);
      }
    }
    __syncwarp();  // rows fully consumed before the next iteration overwrites them
  }
}

}  // namespace dgq

extern "C" dgq_status dgq_quantize_act(const dgq_groups* g, int timestep, int mode, int layout, const void* X,
                                       int64_t M, int64_t ld, void* Xq, float* dyn_scale, int32_t* dyn_zp,
                                       void* stream) {
  using namespace dgq;
  if (!g || !X || !Xq || M <= 0 || ld < g->C) return DGQ_ERR_INVALID_ARG;
  if (mode != DGQ_MODE_STATIC && mode != DGQ_MODE_DYNAMIC_TOKEN) return DGQ_ERR_INVALID_ARG;
  if (layout != DGQ_CODES_U8 && layout != DGQ_CODES_S8_CENTRED) return DGQ_ERR_INVALID_ARG;
  if (timestep < 0 || timestep >= g->T) return DGQ_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(Xq) || (ld % 8) != 0) return DGQ_ERR_ALIGNMENT;
  if ((g->C % 8) != 0) return DGQ_ERR_UNSUPPORTED;
  const int L = (1 << g->bits) - 1;
  const size_t trow = (size_t)timestep * g->R * g->G;
  if (mode == DGQ_MODE_STATIC) {
    if (!g->filled[timestep]) return DGQ_ERR_NOT_CALIBRATED;
    if (layout == DGQ_CODES_S8_CENTRED)
      for (int i = 0; i < g->R * g->G; ++i)
        if (g->zp[trow + i] > 128 || g->zp[trow + i] < L - 127) return DGQ_ERR_UNSUPPORTED;
  } else {
    if (!dyn_scale || !dyn_zp) return DGQ_ERR_INVALID_ARG;
    if (layout == DGQ_CODES_S8_CENTRED) return DGQ_ERR_UNSUPPORTED;
  }
  QuantArgs a;
  a.X = (const __half*)X;
  a.Xq = (uint8_t*)Xq;
  a.M = M;
  a.ld = ld;
  a.C = g->C;
  a.K_pad = g->K_pad;
  a.G = g->G;
  a.P = g->P;
  a.bits = g->bits;
  a.dynamic = (mode == DGQ_MODE_DYNAMIC_TOKEN);
  a.centred = (layout == DGQ_CODES_S8_CENTRED);
  a.perm = g->d_perm;
  a.chunk_group = g->d_chunk_group;
  a.row_group = g->d_row_group;
  a.inv_scale = g->d_inv_scale + trow;
  a.zp = g->d_zp + trow;
  a.dyn_scale = dyn_scale;
  a.dyn_zp = dyn_zp;
  const int n_chunks = g->K_pad / 16;
  const int rpw = (g->C <= 1280) ? 2 : 1;
  a.rows_per_warp = rpw;
  const int head = (g->K_pad * 2 + n_chunks + 15) & ~15;
  const int warp_bytes = ((rpw * g->C * 2 + 15) & ~15) + rpw * g->G * 16;
  const size_t smem = (size_t)head + (size_t)QA_WARPS * warp_bytes;
  if (smem > 200 * 1024) return DGQ_ERR_UNSUPPORTED;
  static bool attr_set[64] = {false};
  int dev = 0;
  DGQ_CUDA_OK(cudaGetDevice(&dev));
  if (dev >= 64 || !attr_set[dev]) {
    DGQ_CUDA_OK(cudaFuncSetAttribute(quantize_act_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 200 * 1024));
    if (dev < 64) attr_set[dev] = true;
  }
  const int64_t n_ctas = (M + (int64_t)QA_WARPS * rpw - 1) / ((int64_t)QA_WARPS * rpw);
  const int grid = (int)std::min<int64_t>(n_ctas, 148 * 8);
  quantize_act_kernel<<<grid, QA_THREADS, smem, (cudaStream_t)stream>>>(a);
  g_launches += 1;
  DGQ_CUDA_OK(cudaGetLastError());
  return DGQ_OK;
}
